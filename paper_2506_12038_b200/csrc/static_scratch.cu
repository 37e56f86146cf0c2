// lcd_lut_linear_static: the M <= 16 lookup with its integer scratch inside the library instead of in a buffer
// the caller allocates.  The LCD paper has no counterpart of this entry point; it exists for callers that
// cannot allocate device memory themselves (see include/lcd.h).
#include <cuda_runtime.h>

#include <mutex>

#include "common.h"

namespace lcd {
namespace {

// The scratch itself: part of the library's device image, so every GPU that loads the library holds these
// bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[LCD_STATIC_SCRATCH_BYTES];

// g_static_scratch names a host-side handle here, not device memory: the address a kernel may use has to be
// asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

lcd_status static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return LCD_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return LCD_OK;
}

}  // namespace
}  // namespace lcd

using namespace lcd;

extern "C" lcd_status lcd_lut_linear_static(const void* packed_weights_dev, const void* header_host,
                                            const uint8_t* act_idx, const float* act_scale, int64_t M, float* y,
                                            int64_t ldy, lcd_algo algo, int32_t* status_word_dev,
                                            void* cuda_stream) {
  if (!packed_weights_dev || !header_host || !act_idx || !act_scale || !y || M < 1) return LCD_ERR_INVALID_ARG;
  if (algo != LCD_ALGO_AUTO && algo != LCD_ALGO_REGISTER_LUT && algo != LCD_ALGO_BUCKET_LUT) return LCD_ERR_UNSUPPORTED;
  if (M > 16) return LCD_ERR_UNSUPPORTED;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  if (ldy < (int64_t)h.N) return LCD_ERR_INVALID_ARG;
  auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
  if (misaligned(packed_weights_dev, 256) || misaligned(act_idx, 16) || misaligned(act_scale, 4) || misaligned(y, 4))
    return LCD_ERR_INVALID_ARG;
  Problem p;
  const uint8_t* blob = static_cast<const uint8_t*>(packed_weights_dev);
  p.tiles = blob + h.index_offset;
  p.codebook = reinterpret_cast<const uint16_t*>(blob + h.codebook_offset);
  p.N = (int64_t)h.N;
  p.K = (int64_t)h.K;
  p.K_pad = (int64_t)h.K_pad;
  p.N_pad = (int64_t)round_up_u64(h.N, kPairRows);
  p.bits = (int)h.bits;
  p.C = (int)h.C;
  p.act_idx = act_idx;
  p.act_scale = act_scale;
  p.M = M;
  p.y = y;
  p.ldy = ldy;
  const lcd_algo family = algo == LCD_ALGO_AUTO ? LCD_ALGO_REGISTER_LUT : algo;
  const size_t need = lut_gemv_workspace_bytes(&p, 1, family);
  if (need > (size_t)LCD_STATIC_SCRATCH_BYTES) return LCD_ERR_BUFFER_TOO_SMALL;   // layer too large for the built-in scratch
  void* scratch = nullptr;
  const lcd_status st = static_scratch_address(&scratch);
  if (st != LCD_OK) return st;
  // every call shares the array and finds whatever the previous one left: the kernel wants zeros
  const cudaError_t e = cudaMemsetAsync(scratch, 0, need, static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return launch_lut_gemv(&p, 1, family, scratch, need, status_word_dev, cuda_stream);
}
