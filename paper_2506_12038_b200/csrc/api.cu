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

static lcd_algo resolve_algo(const Problem& p, lcd_algo algo) {
  if (algo != LCD_ALGO_AUTO) return algo;
  if (p.M <= 16) return resolve_small_m(&p, 1, algo);
  return kHaveDenseTc ? LCD_ALGO_DENSE_TC : LCD_ALGO_REFERENCE;
}

// LCD_ALGO_AUTO between 17 and 32 tokens on long rows: two launches of the register-table kernel (16 tokens, then
// the rest) beat the tensor-core kernel, whose 128-token tile is mostly empty there and whose time grows with the
// row length (measured on 4096 x 11008: 31.5 vs 41.0 us at M = 17, 46 vs 41 at M = 32 with 2-bit indices, 28.5 vs
// 49 and 39 vs 49 with 3-bit ones; on rows of 4096 columns the two are within 5 % at M = 17 and the tensor-core
// kernel wins from M = 24 on; from M = 64 it wins everywhere by 2 to 8 times).
static bool two_chunks(const Problem& p, lcd_algo algo) {
  return algo == LCD_ALGO_AUTO && p.act_bits == 4 && p.M > 16 && p.M <= 32 && p.K_pad >= 8192;
}

static bool small_m_family(lcd_algo a) {
  return a == LCD_ALGO_REGISTER_LUT || a == LCD_ALGO_BUCKET_LUT || a == LCD_ALGO_TC_LUT || a == LCD_ALGO_SHARED_BUCKET;
}

// Fills everything of a Problem that follows from the blob header and the call's pointers.
static lcd_status make_problem(const void* packed_weights_dev, const void* header_host, const uint8_t* act_idx,
                               const float* act_scale, int64_t M, float* y, int64_t ldy, Problem* p) {
  if (!packed_weights_dev || !header_host || !act_idx || !act_scale || !y || M < 1) return LCD_ERR_INVALID_ARG;
  Header h;
  if (!parse_header(header_host, &h)) return LCD_ERR_BAD_BLOB;
  if (ldy < (int64_t)h.N || M > (1LL << 21)) return LCD_ERR_INVALID_ARG;
  // exact int32 sums of table byte x level: |sum| <= 128 * 8 * K_pad with 4-bit levels (128 * 128 with 8-bit ones,
  // checked where those are accepted)
  if (h.K_pad >= (1ull << 21)) return LCD_ERR_UNSUPPORTED;
  if (!aligned(packed_weights_dev, 256) || !aligned(act_idx, 16) || !aligned(act_scale, 4) || !aligned(y, 4))
    return LCD_ERR_INVALID_ARG;
  const uint8_t* blob = static_cast<const uint8_t*>(packed_weights_dev);
  p->tiles = blob + h.index_offset;
  p->codebook = reinterpret_cast<const uint16_t*>(blob + h.codebook_offset);
  p->N = (int64_t)h.N;
  p->K = (int64_t)h.K;
  p->K_pad = (int64_t)h.K_pad;
  p->N_pad = (int64_t)round_up_u64(h.N, kPairRows);
  p->bits = (int)h.bits;
  p->C = (int)h.C;
  p->act_idx = act_idx;
  p->act_scale = act_scale;
  p->M = M;
  p->y = y;
  p->ldy = ldy;
  return LCD_OK;
}

// Sizes only (no pointers needed): the Problem a header and a token count describe.
static bool shape_problem(const void* header_host, int64_t M, Problem* p) {
  Header h;
  if (!parse_header(header_host, &h)) return false;
  *p = Problem{};
  p->N = (int64_t)h.N;
  p->K = (int64_t)h.K;
  p->K_pad = (int64_t)h.K_pad;
  p->N_pad = (int64_t)round_up_u64(h.N, kPairRows);
  p->bits = (int)h.bits;
  p->C = (int)h.C;
  p->M = M;
  return true;
}

static lcd_status workspace_for(const Problem& p, lcd_algo algo, size_t* bytes) {
  if (two_chunks(p, algo)) {
    Problem first = p;
    first.M = 16;
    *bytes = lut_gemv_workspace_bytes(&first, 1, LCD_ALGO_REGISTER_LUT);
    return LCD_OK;
  }
  const lcd_algo resolved = resolve_algo(p, algo);
  switch (resolved) {
    case LCD_ALGO_REFERENCE:
      *bytes = 0;
      return LCD_OK;
    case LCD_ALGO_REGISTER_LUT:
    case LCD_ALGO_BUCKET_LUT:
    case LCD_ALGO_TC_LUT:
    case LCD_ALGO_SHARED_BUCKET:
      if (p.M > 16) return LCD_ERR_UNSUPPORTED;
      if (resolved == LCD_ALGO_SHARED_BUCKET && !lut_smem_supported(&p, 1)) return LCD_ERR_UNSUPPORTED;
      *bytes = lut_gemv_workspace_bytes(&p, 1, resolved);
      return LCD_OK;
    case LCD_ALGO_DENSE_TC:
    case LCD_ALGO_DENSE_F16:
      *bytes = dense_tc_workspace_bytes(p.M, p.K_pad);
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
  if (act_bits != LCD_ACT_BITS && act_bits != 8) return LCD_ERR_UNSUPPORTED;
  if (!aligned(x_fp16, 2) || !aligned(act_scale, 4) || (inv_smooth && !aligned(inv_smooth, 4)))
    return LCD_ERR_INVALID_ARG;
  if (act_bits == 8)
    return launch_smooth_quantize8(x_fp16, M, K, ldx, inv_smooth, static_scale, reinterpret_cast<int8_t*>(act_idx),
                                   act_scale, cuda_stream);
  return launch_smooth_quantize(x_fp16, M, K, ldx, inv_smooth, static_scale, act_idx, act_scale, cuda_stream);
}

extern "C" lcd_status lcd_smooth_quantize_act_batch(const lcd_act_problem* problems, int count, int act_bits,
                                                    void* cuda_stream) {
  if (!problems || count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  if (act_bits != LCD_ACT_BITS && act_bits != 8) return LCD_ERR_UNSUPPORTED;
  for (int i = 0; i < count; ++i) {
    const lcd_act_problem& q = problems[i];
    if (!q.x_fp16 || !q.act_idx || !q.act_scale || q.M < 1 || q.K < 1 || q.ldx < q.K || q.M > 0x7fffffffLL)
      return LCD_ERR_INVALID_ARG;
    if (!aligned(q.x_fp16, 2) || !aligned(q.act_scale, 4) || (q.inv_smooth && !aligned(q.inv_smooth, 4)))
      return LCD_ERR_INVALID_ARG;
  }
  if (act_bits == 8) return launch_smooth_quantize8_batch(problems, count, cuda_stream);
  return launch_smooth_quantize_batch(problems, count, cuda_stream);
}

extern "C" lcd_status lcd_lut_linear_workspace_bytes(const void* header_host, int64_t M, lcd_algo algo,
                                                     size_t* bytes) {
  if (!header_host || !bytes || M < 1) return LCD_ERR_INVALID_ARG;
  Problem p;
  if (!shape_problem(header_host, M, &p)) return LCD_ERR_BAD_BLOB;
  return workspace_for(p, algo, bytes);
}

extern "C" lcd_status lcd_lut_linear(const void* packed_weights_dev, const void* header_host,
                                     const uint8_t* act_idx, const float* act_scale, int64_t M, float* y,
                                     int64_t ldy, lcd_algo algo, void* workspace, size_t workspace_bytes,
                                     int32_t* status_word_dev, void* cuda_stream) {
  Problem p;
  lcd_status st = make_problem(packed_weights_dev, header_host, act_idx, act_scale, M, y, ldy, &p);
  if (st != LCD_OK) return st;
  size_t need = 0;
  st = workspace_for(p, algo, &need);
  if (st != LCD_OK) return st;
  if (need > 0 && (!workspace || workspace_bytes < need)) return LCD_ERR_BUFFER_TOO_SMALL;
  if (need > 0 && !aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
  if (two_chunks(p, algo)) {
    // the second launch touches the scratch only after the first one has finished (stream order, dependency wait)
    Problem part = p;
    part.M = 16;
    st = launch_lut_gemv(&part, 1, LCD_ALGO_REGISTER_LUT, workspace, workspace_bytes, status_word_dev, cuda_stream);
    if (st != LCD_OK) return st;
    part.M = p.M - 16;
    part.act_idx = p.act_idx + 16 * (p.K_pad / 2);
    part.act_scale = p.act_scale + 16;
    part.y = p.y + 16 * p.ldy;
    return launch_lut_gemv(&part, 1, LCD_ALGO_REGISTER_LUT, workspace, workspace_bytes, status_word_dev, cuda_stream);
  }
  const lcd_algo resolved = resolve_algo(p, algo);
  switch (resolved) {
    case LCD_ALGO_REFERENCE:
      return launch_reference(p, cuda_stream);
    case LCD_ALGO_REGISTER_LUT:
    case LCD_ALGO_BUCKET_LUT:
    case LCD_ALGO_TC_LUT:
    case LCD_ALGO_SHARED_BUCKET:
      return launch_lut_gemv(&p, 1, resolved, workspace, workspace_bytes, status_word_dev, cuda_stream);
    case LCD_ALGO_DENSE_TC:
    case LCD_ALGO_DENSE_F16:
      return launch_dense_tc(p, resolved == LCD_ALGO_DENSE_F16, workspace, workspace_bytes, status_word_dev, cuda_stream);
    default:
      return LCD_ERR_INVALID_ARG;
  }
}

static lcd_status batch_algo(const lcd_linear_problem* problems, int count, lcd_algo algo) {
  if (!problems || count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  if (algo != LCD_ALGO_AUTO && !small_m_family(algo)) return LCD_ERR_UNSUPPORTED;
  for (int i = 0; i < count; ++i)
    if (problems[i].M < 1 || problems[i].M > 16) return problems[i].M < 1 ? LCD_ERR_INVALID_ARG : LCD_ERR_UNSUPPORTED;
  return LCD_OK;
}
// The family a grouped call runs: the caller's, or the library's choice for these shapes.
static lcd_status batch_family(const Problem* p, int count, lcd_algo algo, lcd_algo* resolved) {
  *resolved = resolve_small_m(p, count, algo);
  if (*resolved == LCD_ALGO_SHARED_BUCKET && !lut_smem_supported(p, count)) return LCD_ERR_UNSUPPORTED;
  return LCD_OK;
}

extern "C" lcd_status lcd_lut_linear_batch_workspace_bytes(const lcd_linear_problem* problems, int count,
                                                           lcd_algo algo, size_t* bytes) {
  lcd_algo resolved;
  lcd_status st = batch_algo(problems, count, algo);
  if (st != LCD_OK) return st;
  if (!bytes) return LCD_ERR_INVALID_ARG;
  Problem p[LCD_MAX_BATCH];
  for (int i = 0; i < count; ++i) {
    if (!problems[i].header_host) return LCD_ERR_INVALID_ARG;
    if (!shape_problem(problems[i].header_host, problems[i].M, &p[i])) return LCD_ERR_BAD_BLOB;
    if (p[i].bits != p[0].bits) return LCD_ERR_UNSUPPORTED;
  }
  st = batch_family(p, count, algo, &resolved);
  if (st != LCD_OK) return st;
  *bytes = lut_gemv_workspace_bytes(p, count, resolved);
  return LCD_OK;
}

extern "C" lcd_status lcd_lut_linear_batch_resolve(const lcd_linear_problem* problems, int count, lcd_algo algo,
                                                   lcd_algo* resolved) {
  lcd_status st = batch_algo(problems, count, algo);
  if (st != LCD_OK) return st;
  if (!resolved) return LCD_ERR_INVALID_ARG;
  Problem p[LCD_MAX_BATCH];
  for (int i = 0; i < count; ++i) {
    if (!problems[i].header_host) return LCD_ERR_INVALID_ARG;
    if (!shape_problem(problems[i].header_host, problems[i].M, &p[i])) return LCD_ERR_BAD_BLOB;
    if (p[i].bits != p[0].bits) return LCD_ERR_UNSUPPORTED;
  }
  return batch_family(p, count, algo, resolved);
}

extern "C" lcd_status lcd_lut_linear_batch(const lcd_linear_problem* problems, int count, lcd_algo algo,
                                           void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                           void* cuda_stream) {
  lcd_algo resolved;
  lcd_status st = batch_algo(problems, count, algo);
  if (st != LCD_OK) return st;
  Problem p[LCD_MAX_BATCH];
  for (int i = 0; i < count; ++i) {
    const lcd_linear_problem& q = problems[i];
    st = make_problem(q.packed_weights_dev, q.header_host, q.act_idx, q.act_scale, q.M, q.y, q.ldy, &p[i]);
    if (st != LCD_OK) return st;
    if (p[i].bits != p[0].bits) return LCD_ERR_UNSUPPORTED;
  }
  st = batch_family(p, count, algo, &resolved);
  if (st != LCD_OK) return st;
  const size_t need = lut_gemv_workspace_bytes(p, count, resolved);
  if (!workspace || workspace_bytes < need) return LCD_ERR_BUFFER_TOO_SMALL;
  if (!aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
  return launch_lut_gemv(p, count, resolved, workspace, workspace_bytes, status_word_dev, cuda_stream);
}

extern "C" lcd_status lcd_lut_linear_batch_act8(const lcd_linear_problem* problems, int count, lcd_algo algo,
                                           void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                           void* cuda_stream) {
  lcd_algo resolved;
  lcd_status st = batch_algo(problems, count, algo);
  if (st != LCD_OK) return st;
  Problem p[LCD_MAX_BATCH];
  for (int i = 0; i < count; ++i) {
    const lcd_linear_problem& q = problems[i];
    st = make_problem(q.packed_weights_dev, q.header_host, q.act_idx, q.act_scale, q.M, q.y, q.ldy, &p[i]);
    if (st != LCD_OK) return st;
    if (p[i].bits != p[0].bits) return LCD_ERR_UNSUPPORTED;
    p[i].act_bits = 8;
    if (p[i].K_pad >= (1LL << 17)) return LCD_ERR_UNSUPPORTED;   // int32 sums could overflow
  }
  st = batch_family(p, count, algo, &resolved);
  if (st != LCD_OK) return st;
  const size_t need = lut_gemv_workspace_bytes(p, count, resolved);
  if (!workspace || workspace_bytes < need) return LCD_ERR_BUFFER_TOO_SMALL;
  if (!aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
  return launch_lut_gemv(p, count, resolved, workspace, workspace_bytes, status_word_dev, cuda_stream);
}

extern "C" lcd_status lcd_lut_linear_act8(const void* packed_weights_dev, const void* header_host, const int8_t* act_q,
                                          const float* act_scale, int64_t M, float* y, int64_t ldy, lcd_algo algo,
                                          void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                          void* cuda_stream) {
  Problem p;
  lcd_status st = make_problem(packed_weights_dev, header_host, reinterpret_cast<const uint8_t*>(act_q), act_scale, M,
                               y, ldy, &p);
  if (st != LCD_OK) return st;
  p.act_bits = 8;
  // int32 sums of table byte x level: |sum| <= 128 * 128 * K_pad must stay below 2^31
  if (p.K_pad >= (1LL << 17)) return LCD_ERR_UNSUPPORTED;
  size_t need = 0;
  st = workspace_for(p, algo, &need);
  if (st != LCD_OK) return st;
  if (need > 0 && (!workspace || workspace_bytes < need)) return LCD_ERR_BUFFER_TOO_SMALL;
  if (need > 0 && !aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
  const lcd_algo resolved = resolve_algo(p, algo);
  switch (resolved) {
    case LCD_ALGO_REFERENCE:
      return launch_reference(p, cuda_stream);
    case LCD_ALGO_REGISTER_LUT:
    case LCD_ALGO_BUCKET_LUT:
    case LCD_ALGO_TC_LUT:
      return launch_lut_gemv(&p, 1, resolved, workspace, workspace_bytes, status_word_dev, cuda_stream);
    case LCD_ALGO_DENSE_TC:
      return launch_dense_tc(p, false, workspace, workspace_bytes, status_word_dev, cuda_stream);
    case LCD_ALGO_DENSE_F16:
    case LCD_ALGO_SHARED_BUCKET:      // the shared-memory tables hold sums of four 4-bit levels per byte
      return LCD_ERR_UNSUPPORTED;
    default:
      return LCD_ERR_INVALID_ARG;
  }
}

// Levels and scales of the many-token form of the fused call inside its workspace: per problem M x K_pad signed
// bytes, then M scales, each rounded up to 256 bytes.
static size_t fused_dense_levels_bytes(const Problem& p) { return (size_t)round_up_u64((uint64_t)p.M * p.K_pad, 256); }
static size_t fused_dense_bytes(const Problem& p) {
  return fused_dense_levels_bytes(p) + (size_t)round_up_u64((uint64_t)p.M * sizeof(float), 256);
}

static lcd_status fused_problems(const lcd_fused_problem* problems, int count, lcd_algo algo, bool pointers,
                                 Problem* p, lcd_algo* resolved) {
  if (!problems || count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  if (algo != LCD_ALGO_AUTO && algo != LCD_ALGO_REGISTER_LUT && algo != LCD_ALGO_BUCKET_LUT &&
      algo != LCD_ALGO_SHARED_BUCKET && algo != LCD_ALGO_DENSE_TC)
    return LCD_ERR_UNSUPPORTED;
  // either every problem has at most 16 tokens (one lookup launch that transforms its inputs itself) or every
  // problem has more than 16 (one transformation launch, then the tensor-core kernel per problem)
  bool many = false;
  for (int i = 0; i < count; ++i) many = many || (problems[i].M > 16);
  for (int i = 0; i < count; ++i) {
    const lcd_fused_problem& q = problems[i];
    if (q.M < 1 || !q.header_host) return LCD_ERR_INVALID_ARG;
    if (many ? (q.M <= 16 || (algo != LCD_ALGO_AUTO && algo != LCD_ALGO_DENSE_TC)) : algo == LCD_ALGO_DENSE_TC)
      return LCD_ERR_UNSUPPORTED;
    if (!shape_problem(q.header_host, q.M, &p[i])) return LCD_ERR_BAD_BLOB;
    if (many && p[i].K_pad >= (1 << 21)) return LCD_ERR_UNSUPPORTED;      // the int32 sums of the planes could overflow
    if (p[i].bits != p[0].bits) return LCD_ERR_UNSUPPORTED;
    p[i].act_bits = 16;
    if (!pointers) continue;
    if (!q.packed_weights_dev || !q.x_fp16 || !q.y || q.ldx < p[i].K || q.ldy < p[i].N) return LCD_ERR_INVALID_ARG;
    if (!aligned(q.packed_weights_dev, 256) || !aligned(q.x_fp16, 2) || !aligned(q.y, 4) ||
        (q.inv_smooth && !aligned(q.inv_smooth, 4)))
      return LCD_ERR_INVALID_ARG;
    Header h;
    parse_header(q.header_host, &h);
    const uint8_t* blob = static_cast<const uint8_t*>(q.packed_weights_dev);
    p[i].tiles = blob + h.index_offset;
    p[i].codebook = reinterpret_cast<const uint16_t*>(blob + h.codebook_offset);
    p[i].x_fp16 = q.x_fp16;
    p[i].ldx = q.ldx;
    p[i].inv_smooth = q.inv_smooth;
    p[i].y = q.y;
    p[i].ldy = q.ldy;
  }
  if (many) {
    *resolved = LCD_ALGO_DENSE_TC;
    return LCD_OK;
  }
  return batch_family(p, count, algo, resolved);
}

extern "C" lcd_status lcd_linear_fused_batch_workspace_bytes(const lcd_fused_problem* problems, int count,
                                                             lcd_algo algo, size_t* bytes) {
  Problem p[LCD_MAX_BATCH];
  lcd_algo resolved;
  const lcd_status st = fused_problems(problems, count, algo, false, p, &resolved);
  if (st != LCD_OK) return st;
  if (!bytes) return LCD_ERR_INVALID_ARG;
  if (resolved == LCD_ALGO_DENSE_TC) {
    size_t total = 0;
    for (int i = 0; i < count; ++i) total += fused_dense_bytes(p[i]);
    *bytes = total;
    return LCD_OK;
  }
  *bytes = lut_gemv_workspace_bytes(p, count, resolved);
  return LCD_OK;
}

extern "C" lcd_status lcd_linear_fused_batch(const lcd_fused_problem* problems, int count, lcd_algo algo,
                                             void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                             void* cuda_stream) {
  Problem p[LCD_MAX_BATCH];
  lcd_algo resolved;
  lcd_status st = fused_problems(problems, count, algo, true, p, &resolved);
  if (st != LCD_OK) return st;
  if (resolved == LCD_ALGO_DENSE_TC) {
    // Many tokens: ONE launch transforms the inputs of all problems (Section 4.1, the operation sequence of
    // lcd_smooth_quantize_act) and writes the levels as the signed bytes the tensor-core kernel reads, in its order:
    // no packed 4-bit copy, no expansion pass.  Then that kernel, once per problem.
    size_t need = 0;
    for (int i = 0; i < count; ++i) need += fused_dense_bytes(p[i]);
    if (!workspace || workspace_bytes < need) return LCD_ERR_BUFFER_TOO_SMALL;
    if (!aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
    lcd_act_problem acts[LCD_MAX_BATCH];
    uint8_t* at = static_cast<uint8_t*>(workspace);
    for (int i = 0; i < count; ++i) {
      acts[i].x_fp16 = p[i].x_fp16;
      acts[i].M = p[i].M;
      acts[i].K = p[i].K;
      acts[i].ldx = p[i].ldx;
      acts[i].inv_smooth = p[i].inv_smooth;
      acts[i].static_scale = nullptr;
      acts[i].act_idx = at;
      acts[i].act_scale = reinterpret_cast<float*>(at + fused_dense_levels_bytes(p[i]));
      at += fused_dense_bytes(p[i]);
    }
    st = launch_smooth_quantize_dense_levels(acts, count, p[0].bits, cuda_stream);
    if (st != LCD_OK) return st;
    for (int i = 0; i < count; ++i) {
      p[i].act_bits = 4;
      p[i].act_idx = acts[i].act_idx;
      p[i].act_scale = acts[i].act_scale;
      p[i].dense_levels = true;
      st = launch_dense_tc(p[i], false, nullptr, 0, status_word_dev, cuda_stream);
      if (st != LCD_OK) return st;
    }
    return LCD_OK;
  }
  const size_t need = lut_gemv_workspace_bytes(p, count, resolved);
  if (!workspace || workspace_bytes < need) return LCD_ERR_BUFFER_TOO_SMALL;
  if (!aligned(workspace, 256)) return LCD_ERR_INVALID_ARG;
  return launch_lut_gemv(p, count, resolved, workspace, workspace_bytes, status_word_dev, cuda_stream);
}

extern "C" lcd_status lcd_smoothing_search_workspace_bytes(int64_t T, int64_t K, int n_alphas, size_t* bytes) {
  if (!bytes || T < 1 || K < 1 || n_alphas < 1 || n_alphas > 64) return LCD_ERR_INVALID_ARG;
  if (T > 0x7fffffffLL) return LCD_ERR_INVALID_ARG;
  *bytes = smoothing_search_workspace_bytes(T, K, n_alphas);
  return LCD_OK;
}

extern "C" lcd_status lcd_smoothing_search(const void* x_fp16, int64_t T, int64_t K, int64_t ldx, const float* wmax,
                                           const float* alphas_host, int n_alphas, void* workspace,
                                           size_t workspace_bytes, double* mse, int32_t* best, float* inv_smooth,
                                           void* cuda_stream) {
  if (!x_fp16 || !wmax || !alphas_host || !workspace || !mse || T < 1 || K < 1 || ldx < K) return LCD_ERR_INVALID_ARG;
  if (n_alphas < 1 || n_alphas > 64 || T > 0x7fffffffLL) return LCD_ERR_INVALID_ARG;
  if (!aligned(x_fp16, 2) || !aligned(wmax, 4) || !aligned(workspace, 256) || !aligned(mse, 8) ||
      (best && !aligned(best, 4)) || (inv_smooth && !aligned(inv_smooth, 4)))
    return LCD_ERR_INVALID_ARG;
  if (workspace_bytes < smoothing_search_workspace_bytes(T, K, n_alphas)) return LCD_ERR_BUFFER_TOO_SMALL;
  return launch_smoothing_search(x_fp16, T, K, ldx, wmax, alphas_host, n_alphas, workspace, mse, best, inv_smooth,
                                 cuda_stream);
}

extern "C" lcd_status lcd_reclassify(const uint8_t* idx, const uint16_t* codebook_fp16, const float* delta_w, int64_t N,
                                     int64_t K, int64_t ldw, int C, uint8_t* new_idx, double* delta_c, int32_t* counts,
                                     void* cuda_stream) {
  if (!idx || !codebook_fp16 || !delta_w || !new_idx || !delta_c || !counts) return LCD_ERR_INVALID_ARG;
  if (N < 1 || K < 1 || ldw < K || C < 1 || C > 16 || N > 0x7fffffffLL || K > (1LL << 25)) return LCD_ERR_INVALID_ARG;
  if (!aligned(codebook_fp16, 2) || !aligned(delta_w, 4) || !aligned(delta_c, 8) || !aligned(counts, 4))
    return LCD_ERR_INVALID_ARG;
  return launch_reclassify(idx, codebook_fp16, delta_w, N, K, ldw, C, new_idx, delta_c, counts, cuda_stream);
}

extern "C" lcd_status lcd_dbci_workspace_bytes(int64_t n, int max_centroids, size_t* bytes) {
  if (!bytes || n < 1 || n >= 0x7fffffffLL || max_centroids < 1 || max_centroids > (1 << 24)) return LCD_ERR_INVALID_ARG;
  *bytes = dbci_workspace_bytes(n, max_centroids);
  return LCD_OK;
}

extern "C" lcd_status lcd_dbci(const float* weights, int64_t n, void* workspace, size_t workspace_bytes, float* centroids,
                               int max_centroids, int32_t* labels, float* sorted, lcd_dbci_result* result,
                               void* cuda_stream) {
  if (!weights || !workspace || !centroids || !result) return LCD_ERR_INVALID_ARG;
  if (n < 1 || n >= 0x7fffffffLL || max_centroids < 1 || max_centroids > (1 << 24)) return LCD_ERR_INVALID_ARG;
  if (!aligned(weights, 4) || !aligned(workspace, 256) || !aligned(centroids, 4) || !aligned(result, 8) ||
      (labels && !aligned(labels, 4)) || (sorted && !aligned(sorted, 4)))
    return LCD_ERR_INVALID_ARG;
  if (workspace_bytes < dbci_workspace_bytes(n, max_centroids)) return LCD_ERR_BUFFER_TOO_SMALL;
  return launch_dbci(weights, n, workspace, centroids, max_centroids, labels, sorted, result, cuda_stream);
}

// ---- host-buffer path -------------------------------------------------------------------------------
namespace {
struct HostScratch {
  size_t x_off, idx_off, scale_off, y_off, ws_off, ws_bytes, total;
};
lcd_status host_scratch_layout(const Header& h, int64_t M, HostScratch* s) {
  size_t ws = 0;
  Problem shape;
  if (!shape_problem(&h, M, &shape)) return LCD_ERR_BAD_BLOB;
  lcd_status st = workspace_for(shape, LCD_ALGO_AUTO, &ws);
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
                                      void* scratch, size_t scratch_bytes, int32_t* status_word_dev,
                                      void* cuda_stream) {
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
  // the workspace part was zero-filled by the caller before the first call and is left zero-filled by every call
  st = lcd_lut_linear(packed_weights_dev, header_host, idx, scale, M, y, (int64_t)h.N, LCD_ALGO_AUTO,
                      s.ws_bytes ? base + s.ws_off : nullptr, s.ws_bytes, status_word_dev, cuda_stream);
  if (st != LCD_OK) return st;
  e = cudaMemcpyAsync(y_host, y, (size_t)M * h.N * 4, cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

// ---- host-buffer path, grouped ----------------------------------------------------------------------
namespace {
struct HostBatchLayout {
  size_t x_off[LCD_MAX_BATCH], idx_off[LCD_MAX_BATCH], scale_off[LCD_MAX_BATCH], y_off[LCD_MAX_BATCH];
  size_t x_bytes, y_bytes;      // staging areas (all inputs / all outputs, contiguous)
  size_t ws_off, ws_bytes, total;
};
// Device scratch: | all x (dense, in problem order) | all y (dense, in problem order) | indices | scales | workspace |
lcd_status host_batch_layout(const lcd_host_problem* probs, int count, Problem* shapes, HostBatchLayout* L) {
  if (!probs || count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  size_t o = 0;
  for (int i = 0; i < count; ++i) {
    if (!probs[i].header_host || probs[i].M < 1) return LCD_ERR_INVALID_ARG;
    if (probs[i].M > 16) return LCD_ERR_UNSUPPORTED;
    if (!shape_problem(probs[i].header_host, probs[i].M, &shapes[i])) return LCD_ERR_BAD_BLOB;
    if (shapes[i].bits != shapes[0].bits) return LCD_ERR_UNSUPPORTED;
    L->x_off[i] = o;
    o += (size_t)round_up_u64((uint64_t)probs[i].M * shapes[i].K * 2, 16);
  }
  L->x_bytes = o;
  o = (size_t)round_up_u64(o, 256);
  const size_t y0 = o;
  for (int i = 0; i < count; ++i) {
    L->y_off[i] = o;
    o += (size_t)round_up_u64((uint64_t)probs[i].M * shapes[i].N * 4, 16);
  }
  L->y_bytes = o - y0;
  o = (size_t)round_up_u64(o, 256);
  for (int i = 0; i < count; ++i) {
    L->idx_off[i] = o;
    o += (size_t)round_up_u64((uint64_t)probs[i].M * shapes[i].K_pad / 2, 256);
    L->scale_off[i] = o;
    o += 256;
  }
  L->ws_off = o;
  L->ws_bytes = lut_gemv_workspace_bytes(shapes, count, resolve_small_m(shapes, count, LCD_ALGO_AUTO));
  L->total = o + (size_t)round_up_u64(L->ws_bytes, 256);
  return LCD_OK;
}
}  // namespace

extern "C" lcd_status lcd_linear_host_batch_sizes(const lcd_host_problem* problems, int count, size_t* x_host_bytes,
                                                  size_t* y_host_bytes, size_t* scratch_bytes) {
  Problem shapes[LCD_MAX_BATCH];
  HostBatchLayout L;
  const lcd_status st = host_batch_layout(problems, count, shapes, &L);
  if (st != LCD_OK) return st;
  if (x_host_bytes) *x_host_bytes = L.x_bytes;
  if (y_host_bytes) *y_host_bytes = L.y_bytes;
  if (scratch_bytes) *scratch_bytes = L.total;
  return LCD_OK;
}

extern "C" lcd_status lcd_linear_host_batch(const lcd_host_problem* problems, int count, const void* x_host_all,
                                            void* y_host_all, void* scratch, size_t scratch_bytes,
                                            int32_t* status_word_dev, void* cuda_stream) {
  if (!x_host_all || !y_host_all || !scratch) return LCD_ERR_INVALID_ARG;
  Problem shapes[LCD_MAX_BATCH];
  HostBatchLayout L;
  lcd_status st = host_batch_layout(problems, count, shapes, &L);
  if (st != LCD_OK) return st;
  if (scratch_bytes < L.total) return LCD_ERR_BUFFER_TOO_SMALL;
  if (!aligned(scratch, 256)) return LCD_ERR_INVALID_ARG;
  uint8_t* base = static_cast<uint8_t*>(scratch);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(base, x_host_all, L.x_bytes, cudaMemcpyHostToDevice, stream);   // one copy in
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  // A small y goes straight into the caller's buffer when the device can address it (pinned, mapped host memory): the
  // kernels' stores cross the bus themselves and there is no copy out (7B layer, one token, 170 KB: 46 instead of
  // 59 us end to end).  Larger outputs are copied: the kernels store 32-byte pieces, which the bus takes badly
  // (16 tokens, 2.7 MB: 193 instead of 141 us).
  constexpr size_t kDirectOutputBytes = 512 << 10;
  uint8_t* y_direct = nullptr;
  if (L.y_bytes <= kDirectOutputBytes) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, y_host_all) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
      y_direct = static_cast<uint8_t*>(attr.devicePointer);
    else
      (void)cudaGetLastError();
  }
  lcd_act_problem acts[LCD_MAX_BATCH];
  Problem p[LCD_MAX_BATCH];
  for (int i = 0; i < count; ++i) {
    acts[i].x_fp16 = base + L.x_off[i];
    acts[i].M = problems[i].M;
    acts[i].K = shapes[i].K;
    acts[i].ldx = shapes[i].K;
    acts[i].inv_smooth = problems[i].inv_smooth;
    acts[i].static_scale = nullptr;
    acts[i].act_idx = base + L.idx_off[i];
    acts[i].act_scale = reinterpret_cast<float*>(base + L.scale_off[i]);
    st = make_problem(problems[i].packed_weights_dev, problems[i].header_host, acts[i].act_idx, acts[i].act_scale,
                      problems[i].M,
                      reinterpret_cast<float*>(y_direct ? y_direct + (L.y_off[i] - L.y_off[0]) : base + L.y_off[i]),
                      shapes[i].N, &p[i]);
    if (st != LCD_OK) return st;
  }
  // Single tokens: the lookup kernel does the input transformation itself (one launch less, the levels are never
  // written to memory).  With more tokens every CTA would repeat the transformation of all of them, which costs
  // more than the separate launch (measured), so that launch stays.
  bool single_tokens = true;
  for (int i = 0; i < count; ++i) single_tokens = single_tokens && problems[i].M == 1;
  if (single_tokens) {
    for (int i = 0; i < count; ++i) {
      p[i].act_bits = 16;
      p[i].x_fp16 = acts[i].x_fp16;
      p[i].ldx = acts[i].ldx;
      p[i].inv_smooth = acts[i].inv_smooth;
    }
  } else {
    st = lcd_smooth_quantize_act_batch(acts, count, LCD_ACT_BITS, cuda_stream);
    if (st != LCD_OK) return st;
  }
  // the workspace part was zero-filled by the caller before the first call and is left zero-filled by every call
  st = launch_lut_gemv(p, count, resolve_small_m(shapes, count, LCD_ALGO_AUTO), base + L.ws_off, L.ws_bytes, status_word_dev,
                       cuda_stream);
  if (st != LCD_OK) return st;
  if (!y_direct) {
    e = cudaMemcpyAsync(y_host_all, base + L.y_off[0], L.y_bytes, cudaMemcpyDeviceToHost, stream);   // one copy out
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  }
  return LCD_OK;
}
