// C ABI: argument checking and dispatch.  The three stages of Section 4 of the LCD paper map to
// lcd_smooth_quantize_act (input transformation) and lcd_lut_linear (bucket table lookup + accumulation).
#include <cuda_runtime.h>

#include <cstring>
#include <string>

#include "common.h"

namespace lcd {

static thread_local std::string g_cuda_error;

void set_cuda_error(int err) { g_cuda_error = cudaGetErrorString(static_cast<cudaError_t>(err)); }

static bool aligned(const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a == 0; }

static lcd_algo resolve_algo(const Header& h, int64_t M, lcd_algo algo) {
  if (algo != LCD_ALGO_AUTO) return algo;
  if (M == 1 && h.bits == 2 && kHaveBucketLut) return LCD_ALGO_BUCKET_LUT;
  if (M <= 16) return LCD_ALGO_REGISTER_LUT;
  return kHaveDenseTc ? LCD_ALGO_DENSE_TC : LCD_ALGO_REFERENCE;
}

static lcd_status workspace_for(const Header& h, int64_t M, lcd_algo algo, size_t* bytes) {
  const int64_t n_pad = (int64_t)round_up_u64(h.N, kTileRows);
  switch (resolve_algo(h, M, algo)) {
    case LCD_ALGO_REFERENCE:
    case LCD_ALGO_REGISTER_LUT:
      *bytes = 0;
      return LCD_OK;
    case LCD_ALGO_BUCKET_LUT:
      *bytes = bucket_lut_workspace_bytes(n_pad, (int64_t)h.K_pad);
      return LCD_OK;
    case LCD_ALGO_DENSE_TC:
      *bytes = dense_tc_workspace_bytes(M, (int64_t)h.K_pad);
      return LCD_OK;
    default:
      return LCD_ERR_INVALID_ARG;
  }
}

}  // namespace lcd

using namespace lcd;

extern "C" const char* lcd_status_string(lcd_status s) {
  switch (s) {
    case LCD_OK: return "ok";
    case LCD_ERR_INVALID_ARG: return "invalid argument";
    case LCD_ERR_UNSUPPORTED: return "unsupported";
    case LCD_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case LCD_ERR_INDEX_RANGE: return "weight index out of range";
    case LCD_ERR_BAD_BLOB: return "bad packed-weights blob";
    case LCD_ERR_CUDA: return "CUDA error";
    case LCD_ERR_TIMEOUT: return "device-side wait expired";
  }
  return "unknown status";
}

extern "C" const char* lcd_last_cuda_error(void) { return g_cuda_error.c_str(); }

extern "C" lcd_status lcd_smooth_quantize_act(const void* x_fp16, int64_t M, int64_t K, int64_t ldx,
                                              const float* inv_smooth, const float* static_scale, int act_bits,
                                              uint8_t* act_idx, float* act_scale, void* cuda_stream) {
  if (!x_fp16 || !act_idx || !act_scale || M < 1 || K < 1 || ldx < K) return LCD_ERR_INVALID_ARG;
  if (M > 0x7fffffffLL) return LCD_ERR_INVALID_ARG;
  if (act_bits != LCD_ACT_BITS) return LCD_ERR_UNSUPPORTED;
  if (!aligned(x_fp16, 2) || !aligned(act_scale, 4) || (inv_smooth && !aligned(inv_smooth, 4)))
    return LCD_ERR_INVALID_ARG;
  return launch_smooth_quantize(x_fp16, M, K, ldx, inv_smooth, static_scale, act_idx, act_scale, cuda_stream);
}

extern "C" lcd_status lcd_lut_linear_workspace_bytes(const void* header_host, int64_t M, lcd_algo algo,
                                                     size_t* bytes) {
  if (!header_host || !bytes || M < 1) return LCD_ERR_INVALID_ARG;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  return workspace_for(h, M, algo, bytes);
}

extern "C" lcd_status lcd_lut_linear(const void* packed_weights_dev, const void* header_host,
                                     const uint8_t* act_idx, const float* act_scale, int64_t M, float* y,
                                     int64_t ldy, lcd_algo algo, void* workspace, size_t workspace_bytes,
                                     int32_t* status_word_dev, void* cuda_stream) {
  if (!packed_weights_dev || !header_host || !act_idx || !act_scale || !y || M < 1) return LCD_ERR_INVALID_ARG;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  if (ldy < (int64_t)h.N || M > (1LL << 21)) return LCD_ERR_INVALID_ARG;
  if (!aligned(packed_weights_dev, 256) || !aligned(act_idx, 16) || !aligned(act_scale, 4) || !aligned(y, 4))
    return LCD_ERR_INVALID_ARG;
  size_t need = 0;
  lcd_status st = workspace_for(h, M, algo, &need);
  if (st != LCD_OK) return st;
  if (need > 0 && (!workspace || workspace_bytes < need)) return LCD_ERR_BUFFER_TOO_SMALL;
  if (need > 0 && !aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;

  Problem p;
  const uint8_t* blob = static_cast<const uint8_t*>(packed_weights_dev);
  p.tiles = blob + h.index_offset;
  p.codebook = reinterpret_cast<const uint16_t*>(blob + h.codebook_offset);
  p.N = (int64_t)h.N;
  p.K = (int64_t)h.K;
  p.K_pad = (int64_t)h.K_pad;
  p.N_pad = (int64_t)round_up_u64(h.N, kTileRows);
  p.bits = (int)h.bits;
  p.C = (int)h.C;
  p.act_idx = act_idx;
  p.act_scale = act_scale;
  p.M = M;
  p.y = y;
  p.ldy = ldy;

  switch (resolve_algo(h, M, algo)) {
    case LCD_ALGO_REFERENCE:
      return launch_reference(p, cuda_stream);
    case LCD_ALGO_BUCKET_LUT:
      if (M != 1 || h.bits != 2) return LCD_ERR_UNSUPPORTED;
      return launch_bucket_lut(p, workspace, workspace_bytes, cuda_stream);
    case LCD_ALGO_REGISTER_LUT:
      if (M > 16) return LCD_ERR_UNSUPPORTED;
      return launch_register_lut(p, cuda_stream);
    case LCD_ALGO_DENSE_TC:
      return launch_dense_tc(p, workspace, workspace_bytes, status_word_dev, cuda_stream);
    default:
      return LCD_ERR_INVALID_ARG;
  }
}

// ---- host-buffer path -------------------------------------------------------------------------------
namespace {
struct HostScratch {
  size_t x_off, idx_off, scale_off, y_off, ws_off, ws_bytes, total;
};
lcd_status host_scratch_layout(const Header& h, int64_t M, HostScratch* s) {
  size_t ws = 0;
  lcd_status st = workspace_for(h, M, LCD_ALGO_AUTO, &ws);
  if (st != LCD_OK) return st;
  size_t o = 0;
  s->x_off = o;      o += round_up_u64((uint64_t)M * h.K * 2, 256);
  s->idx_off = o;    o += round_up_u64((uint64_t)M * h.K_pad / 2, 256);
  s->scale_off = o;  o += round_up_u64((uint64_t)M * 4, 256);
  s->y_off = o;      o += round_up_u64((uint64_t)M * h.N * 4, 256);
  s->ws_off = o;     o += round_up_u64(ws, 256);
  s->ws_bytes = ws;
  s->total = o;
  return LCD_OK;
}
}  // namespace

extern "C" lcd_status lcd_linear_host_scratch_bytes(const void* header_host, int64_t M, size_t* bytes) {
  if (!header_host || !bytes || M < 1) return LCD_ERR_INVALID_ARG;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  HostScratch s;
  lcd_status st = host_scratch_layout(h, M, &s);
  if (st == LCD_OK) *bytes = s.total;
  return st;
}

extern "C" lcd_status lcd_linear_host(const void* packed_weights_dev, const void* header_host,
                                      const void* x_host_fp16, int64_t M, const float* inv_smooth, float* y_host,
                                      void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!packed_weights_dev || !header_host || !x_host_fp16 || !y_host || !scratch || M < 1)
    return LCD_ERR_INVALID_ARG;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  HostScratch s;
  lcd_status st = host_scratch_layout(h, M, &s);
  if (st != LCD_OK) return st;
  if (scratch_bytes < s.total) return LCD_ERR_BUFFER_TOO_SMALL;
  if (!aligned(scratch, 256)) return LCD_ERR_INVALID_ARG;
  uint8_t* base = static_cast<uint8_t*>(scratch);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(base + s.x_off, x_host_fp16, (size_t)M * h.K * 2, cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  uint8_t* idx = base + s.idx_off;
  float* scale = reinterpret_cast<float*>(base + s.scale_off);
  float* y = reinterpret_cast<float*>(base + s.y_off);
  st = lcd_smooth_quantize_act(base + s.x_off, M, (int64_t)h.K, (int64_t)h.K, inv_smooth, nullptr, LCD_ACT_BITS,
                               idx, scale, cuda_stream);
  if (st != LCD_OK) return st;
  st = lcd_lut_linear(packed_weights_dev, header_host, idx, scale, M, y, (int64_t)h.N, LCD_ALGO_AUTO,
                      s.ws_bytes ? base + s.ws_off : nullptr, s.ws_bytes, nullptr, cuda_stream);
  if (st != LCD_OK) return st;
  e = cudaMemcpyAsync(y_host, y, (size_t)M * h.N * 4, cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}
