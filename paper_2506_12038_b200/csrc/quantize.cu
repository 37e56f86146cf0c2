// Input transformation (Section 4.1 of the LCD paper): smoothing and uniform symmetric quantisation fused
// into one multiply, round to nearest (ties to even), clip to [-8, 7]; emits 4-bit indices a = q + 8 and
// the per-token scale.  Every operation is a single IEEE binary32 operation in the order stated in
// include/lcd.h, so the indices are reproducible bit for bit.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "common.h"

namespace lcd {

constexpr int kQThreads = 1024;   // few tokens: one large CTA per token, everything in registers
constexpr int kQThreadsMany = 256; // many tokens: small CTAs, latency hidden by the number of CTAs
constexpr int kQChunks = 4;    // register-resident path: K <= 8 * kQThreads * kQChunks columns

// a = q + 8 with q = round half to even of v, clipped to the 4-bit symmetric range.  Clipping first gives the same
// level (the bounds are integers), and adding 1.5 * 2^23 + 8 rounds the clipped value to an integer, ties to even,
// in one binary32 addition and leaves q + 8 in the low four bits of the sum: no conversion instructions.
__device__ __forceinline__ uint32_t quant_nibble(float v) {
  const float u = fminf(fmaxf(v, -8.0f), 7.0f);
  return __float_as_uint(__fadd_rn(u, 12582920.0f)) & 0xfu;
}

// Output forms.  kOutNibbles: the levels a = q + 8 packed two per byte, [K_pad / 2] bytes per token (what
// lcd_smooth_quantize_act returns).  kOutBytes / kOutBytes2: the levels q as signed bytes, [K_pad] per token, for
// the tensor-core kernel that follows in the same call: in column order, or in the order in which the 2-bit
// decoder lists the weights of a 32-column quarter (position 16*(c>>4) + 8*(c&1) + 4*((c>>3)&1) + ((c>>1)&3)
// holds column c).
constexpr int kOutNibbles = 0, kOutBytes = 1, kOutBytes2 = 2;

__device__ __forceinline__ uint32_t prmt_q(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
// Eight levels (nibble i of `packed` = a of column k + i, k a multiple of 8) into a token's output row.
template <int OUT, typename Index>
__device__ __forceinline__ void store_levels8(uint8_t* row, Index k, uint32_t packed) {
  if (OUT == kOutNibbles) {
    *reinterpret_cast<uint32_t*>(row + k / 2) = packed;
    return;
  }
  uint32_t e = packed & 0x0f0f0f0fu, o = (packed >> 4) & 0x0f0f0f0fu;     // columns k, k+2, .. / k+1, k+3, ..
  e = (e + 0x78787878u) ^ 0x80808080u;      // per byte a - 8, no carry between bytes
  o = (o + 0x78787878u) ^ 0x80808080u;
  if (OUT == kOutBytes) {
    *reinterpret_cast<uint2*>(row + k) = make_uint2(prmt_q(e, o, 0x5140u), prmt_q(e, o, 0x7362u));
  } else {
    const Index quarter = k & ~(Index)31;
    const int c8 = (int)(k & 31) >> 3;                  // which eight columns of the quarter
    uint8_t* dst = row + quarter + 16 * (c8 >> 1) + 4 * (c8 & 1);
    *reinterpret_cast<uint32_t*>(dst) = e;
    *reinterpret_cast<uint32_t*>(dst + 8) = o;
  }
}
// One level (a = q + 8 of column k).
template <int OUT>
__device__ __forceinline__ void store_level1(uint8_t* row, int64_t k, uint32_t a) {
  const uint8_t q = (uint8_t)((a - 8u) & 0xffu);
  if (OUT == kOutBytes) row[k] = q;
  else {
    const int c = (int)(k & 31);
    row[(k & ~(int64_t)31) + 16 * (c >> 4) + 8 * (c & 1) + 4 * ((c >> 3) & 1) + ((c >> 1) & 3)] = q;
  }
}

// One token per CTA.  VEC: rows are 16-byte aligned and K is a multiple of 8, so each thread handles 8
// consecutive columns per step (one 16-byte load of x, two of inv_smooth, one 4-byte store).
template <bool VEC, int THREADS, int OUT = kOutNibbles>
__device__ __forceinline__ void smooth_quantize_token(const __half* __restrict__ x, int64_t m, int64_t K,
                                                      int64_t K_pad, int64_t ldx,
                                                      const float* __restrict__ inv_smooth,
                                                      const float* __restrict__ static_scale,
                                                      uint8_t* __restrict__ act_idx, float* __restrict__ act_scale) {
  __shared__ float s_red[THREADS / 32];
  __shared__ float s_mult;
  const __half* xr = x + m * ldx;
  uint8_t* out = act_idx + m * (OUT == kOutNibbles ? K_pad / 2 : K_pad);
  const int tid = threadIdx.x;
  const bool is_static = static_scale != nullptr;

  if (!is_static) {
    float amax = 0.0f;
    if (VEC) {
      for (int64_t k = (int64_t)tid * 8; k < K; k += (int64_t)THREADS * 8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xr + k);
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
        float f[8];
        if (inv_smooth) {
          const float4 a = *reinterpret_cast<const float4*>(inv_smooth + k);
          const float4 b = *reinterpret_cast<const float4*>(inv_smooth + k + 4);
          f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) f[i] = 1.0f;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __half22float2(h[i]);
          amax = fmaxf(amax, fabsf(__fmul_rn(v.x, f[2 * i])));
          amax = fmaxf(amax, fabsf(__fmul_rn(v.y, f[2 * i + 1])));
        }
      }
    } else {
      for (int64_t k = tid; k < K; k += THREADS) {
        const float f = inv_smooth ? inv_smooth[k] : 1.0f;
        amax = fmaxf(amax, fabsf(__fmul_rn(__half2float(xr[k]), f)));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = amax;
    __syncthreads();
    if (tid < 32) {
      float v = tid < THREADS / 32 ? s_red[tid] : 0.0f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      if (tid == 0) {
        float sq = 1.0f, r = 0.0f;
        if (v > 0.0f) {
          sq = __fdiv_rn(v, 7.0f);
          r = __fdiv_rn(7.0f, v);
        }
        s_mult = r;
        act_scale[m] = sq;
      }
    }
    __syncthreads();
  } else if (tid == 0) {
    act_scale[m] = *static_scale;
  }
  const float r = is_static ? 1.0f : s_mult;

  if (VEC) {
    for (int64_t k = (int64_t)tid * 8; k < K_pad; k += (int64_t)THREADS * 8) {
      uint32_t packed = 0x88888888u;
      if (k < K) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xr + k);
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
        float f[8];
        if (inv_smooth) {
          const float4 a = *reinterpret_cast<const float4*>(inv_smooth + k);
          const float4 b = *reinterpret_cast<const float4*>(inv_smooth + k + 4);
          f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) f[i] = 1.0f;
        }
        packed = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __half22float2(h[i]);
          float t0 = __fmul_rn(v.x, f[2 * i]), t1 = __fmul_rn(v.y, f[2 * i + 1]);
          if (!is_static) { t0 = __fmul_rn(t0, r); t1 = __fmul_rn(t1, r); }
          const uint32_t a0 = quant_nibble(t0), a1 = quant_nibble(t1);
          packed |= (a0 | (a1 << 4)) << (8 * i);
        }
      }
      store_levels8<OUT>(out, k, packed);
    }
  } else {
    for (int64_t j = tid; j < K_pad / 2; j += THREADS) {
      uint32_t a[2] = {8u, 8u};
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int64_t k = 2 * j + i;
        if (k < K) {
          float t = __fmul_rn(__half2float(xr[k]), inv_smooth ? inv_smooth[k] : 1.0f);
          if (!is_static) t = __fmul_rn(t, r);
          a[i] = quant_nibble(t);
        }
      }
      if (OUT == kOutNibbles) out[j] = (uint8_t)(a[0] | (a[1] << 4));
      else { store_level1<OUT>(out, 2 * j, a[0]); store_level1<OUT>(out, 2 * j + 1, a[1]); }
    }
  }
}

// Same result as smooth_quantize_token<true>, for rows of at most 8 * THREADS * CHUNKS columns: every thread
// keeps its products t_k = x_k * inv_smooth_k in registers between the maximum search and the rounding, so x
// and inv_smooth are read once and all loads are in flight together.
template <int THREADS, int CHUNKS>
__device__ __forceinline__ void smooth_quantize_token_cached(const __half* __restrict__ x, int64_t m, int64_t K,
                                                             int64_t K_pad, int64_t ldx,
                                                             const float* __restrict__ inv_smooth,
                                                             const float* __restrict__ static_scale,
                                                             uint8_t* __restrict__ act_idx,
                                                             float* __restrict__ act_scale) {
  __shared__ float s_red[THREADS / 32];
  __shared__ float s_mult;
  const __half* xr = x + m * ldx;
  uint8_t* out = act_idx + m * (K_pad / 2);
  const int tid = threadIdx.x;
  const bool is_static = static_scale != nullptr;
  float t[CHUNKS][8];
  float amax = 0.0f;
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int64_t k = ((int64_t)c * THREADS + tid) * 8;
    if (k < K) {
      const uint4 raw = *reinterpret_cast<const uint4*>(xr + k);
      const __half2* h = reinterpret_cast<const __half2*>(&raw);
      float f[8];
      if (inv_smooth) {
        const float4 a = *reinterpret_cast<const float4*>(inv_smooth + k);
        const float4 b = *reinterpret_cast<const float4*>(inv_smooth + k + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = 1.0f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 v = __half22float2(h[i]);
        t[c][2 * i] = __fmul_rn(v.x, f[2 * i]);
        t[c][2 * i + 1] = __fmul_rn(v.y, f[2 * i + 1]);
        amax = fmaxf(amax, fmaxf(fabsf(t[c][2 * i]), fabsf(t[c][2 * i + 1])));
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) t[c][i] = 0.0f;
    }
  }
  float r = 1.0f;
  if (!is_static) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = amax;
    __syncthreads();
    if (tid < 32) {
      float v = tid < THREADS / 32 ? s_red[tid] : 0.0f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      if (tid == 0) {
        float sq = 1.0f, rr = 0.0f;
        if (v > 0.0f) {
          sq = __fdiv_rn(v, 7.0f);
          rr = __fdiv_rn(7.0f, v);
        }
        s_mult = rr;
        act_scale[m] = sq;
      }
    }
    __syncthreads();
    r = s_mult;
  } else if (tid == 0) {
    act_scale[m] = *static_scale;
  }
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int64_t k = ((int64_t)c * THREADS + tid) * 8;
    if (k < K_pad) {
      uint32_t packed = 0x88888888u;
      if (k < K) {
        packed = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float u = is_static ? t[c][i] : __fmul_rn(t[c][i], r);
          packed |= quant_nibble(u) << (4 * i);
        }
      }
      *reinterpret_cast<uint32_t*>(out + k / 2) = packed;
    }
  }
}

// The same for many tokens (small CTAs, several per SM): a thread keeps its columns of x as the 16-byte words it
// loaded (four registers per eight columns, so that enough CTAs fit an SM to keep the memory system busy) and forms
// the products x_k * inv_smooth_k twice, with the same single operations, once for the maximum and once for the
// levels; inv_smooth comes from L1 the second time.  Rows of at most 8 * THREADS * CHUNKS columns.
template <int THREADS, int CHUNKS, int OUT = kOutNibbles>
__device__ __forceinline__ void smooth_quantize_token_words(const __half* __restrict__ x, int64_t m, int64_t K64,
                                                            int64_t K_pad64, int64_t ldx,
                                                            const float* __restrict__ inv_smooth,
                                                            const float* __restrict__ static_scale,
                                                            uint8_t* __restrict__ act_idx,
                                                            float* __restrict__ act_scale) {
  __shared__ float s_red[THREADS / 32];
  __shared__ float s_mult;
  const __half* xr = x + m * ldx;
  uint8_t* out = act_idx + m * (OUT == kOutNibbles ? K_pad64 / 2 : K_pad64);
  const int tid = threadIdx.x;
  const bool is_static = static_scale != nullptr;
  const int K = (int)K64, K_pad = (int)K_pad64;        // at most 8 * THREADS * CHUNKS columns: 32-bit column arithmetic
  uint4 raw[CHUNKS];
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int k = (c * THREADS + tid) * 8;
    raw[c] = k < K ? *reinterpret_cast<const uint4*>(xr + k) : make_uint4(0u, 0u, 0u, 0u);
  }
  auto products = [&](int c, int k, float (&t)[8]) {
    const __half2* h = reinterpret_cast<const __half2*>(&raw[c]);
    float f[8];
    if (inv_smooth) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(inv_smooth + k));
      const float4 b = __ldg(reinterpret_cast<const float4*>(inv_smooth + k + 4));
      f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] = 1.0f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 v = __half22float2(h[i]);
      t[2 * i] = __fmul_rn(v.x, f[2 * i]);
      t[2 * i + 1] = __fmul_rn(v.y, f[2 * i + 1]);
    }
  };
  float r = 1.0f;
  if (!is_static) {
    float amax = 0.0f;
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
      const int k = (c * THREADS + tid) * 8;
      if (k < K) {
        float t[8];
        products(c, k, t);
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(t[i]));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = amax;
    __syncthreads();
    if (tid < 32) {
      float v = tid < THREADS / 32 ? s_red[tid] : 0.0f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      if (tid == 0) {
        float sq = 1.0f, rr = 0.0f;
        if (v > 0.0f) {
          sq = __fdiv_rn(v, 7.0f);
          rr = __fdiv_rn(7.0f, v);
        }
        s_mult = rr;
        act_scale[m] = sq;
      }
    }
    __syncthreads();
    r = s_mult;
  } else if (tid == 0) {
    act_scale[m] = *static_scale;
  }
  // static mode: the caller's factors already hold the scale, so the second multiplication is by exactly 1
  const float r_eff = is_static ? 1.0f : r;
#pragma unroll
  for (int c = 0; c < CHUNKS; ++c) {
    const int k = (c * THREADS + tid) * 8;
    if (k < K_pad) {
      // e / o: the levels of columns k, k+2, k+4, k+6 / k+1, k+3, k+5, k+7, one per byte (a = q + 8 for the packed
      // form, q as a signed byte otherwise); padding columns hold level 0
      uint32_t e = OUT == kOutNibbles ? 0x08080808u : 0u, o = e;
      if (k < K) {
        float t[8];
        products(c, k, t);
        uint32_t b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float u = fminf(fmaxf(is_static ? t[i] : __fmul_rn(t[i], r_eff), -8.0f), 7.0f);
          // clipped, then rounded to an integer (ties to even) by one addition: the low byte of the sum is the level
          b[i] = __float_as_uint(__fadd_rn(u, OUT == kOutNibbles ? 12582920.0f : 12582912.0f));
        }
        e = prmt_q(prmt_q(b[0], b[2], 0x0040u), prmt_q(b[4], b[6], 0x0040u), 0x5410u);
        o = prmt_q(prmt_q(b[1], b[3], 0x0040u), prmt_q(b[5], b[7], 0x0040u), 0x5410u);
      }
      if (OUT == kOutNibbles) {
        *reinterpret_cast<uint32_t*>(out + k / 2) = (e & 0x0f0f0f0fu) | ((o & 0x0f0f0f0fu) << 4);
      } else if (OUT == kOutBytes) {
        *reinterpret_cast<uint2*>(out + k) = make_uint2(prmt_q(e, o, 0x5140u), prmt_q(e, o, 0x7362u));
      } else {
        const int c8 = (k & 31) >> 3;                  // which eight columns of the 32-column quarter
        uint8_t* dst = out + (k & ~31) + 16 * (c8 >> 1) + 4 * (c8 & 1);
        *reinterpret_cast<uint32_t*>(dst) = e;
        *reinterpret_cast<uint32_t*>(dst + 8) = o;
      }
    }
  }
}

struct QuantProblem {
  const __half* x;
  const float* inv_smooth;
  const float* static_scale;
  uint8_t* act_idx;
  float* act_scale;
  long long K, K_pad, ldx;
  int cta0;    // tokens of this problem are CTAs [cta0, cta0 + M)
  int vec;
};
struct QuantBatch {
  int count;
  QuantProblem p[LCD_MAX_BATCH];
};

// One CTA per token of every problem of the batch.  CHUNKS > 0: rows of at most 8 * THREADS * CHUNKS columns take the
// register-resident path (the launcher picks the smallest instance that covers the batch's longest row, so that the
// instance's register count, and with it the number of CTAs per SM, fits the rows at hand).
template <int THREADS, int CHUNKS, int OUT = kOutNibbles>
__global__ void __launch_bounds__(THREADS) smooth_quantize_kernel(const __grid_constant__ QuantBatch batch) {
  // This kernel may itself have been started early (programmatic stream serialization): wait for the kernel
  // before it, then let the next one start its own prologue; that one still waits for this grid to finish
  // before it reads the indices.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  int pi = 0;
#pragma unroll 1
  for (int i = 1; i < batch.count; ++i)
    if ((int)blockIdx.x >= batch.p[i].cta0) pi = i;
  const QuantProblem& q = batch.p[pi];
  const int64_t m = (int64_t)blockIdx.x - q.cta0;
  if constexpr (CHUNKS > 0) {
    if (q.vec && q.K_pad <= (long long)8 * THREADS * CHUNKS) {
      if constexpr (THREADS == kQThreads)
        smooth_quantize_token_cached<THREADS, CHUNKS>(q.x, m, q.K, q.K_pad, q.ldx, q.inv_smooth, q.static_scale, q.act_idx,
                                                      q.act_scale);
      else
        smooth_quantize_token_words<THREADS, CHUNKS, OUT>(q.x, m, q.K, q.K_pad, q.ldx, q.inv_smooth, q.static_scale,
                                                          q.act_idx, q.act_scale);
      return;
    }
  }
  if (q.vec)
    smooth_quantize_token<true, THREADS, OUT>(q.x, m, q.K, q.K_pad, q.ldx, q.inv_smooth, q.static_scale, q.act_idx, q.act_scale);
  else
    smooth_quantize_token<false, THREADS, OUT>(q.x, m, q.K, q.K_pad, q.ldx, q.inv_smooth, q.static_scale, q.act_idx, q.act_scale);
}

namespace {

template <int OUT>
cudaError_t launch_small_ctas(const cudaLaunchConfig_t& cfg, long long chunks, const QuantBatch& batch) {
  if (chunks < 1 || chunks > 8) return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 0, OUT>, batch);
  if (chunks <= 2) return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 2, OUT>, batch);
  if (chunks <= 3) return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 3, OUT>, batch);
  if (chunks <= 4) return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 4, OUT>, batch);
  if (chunks <= 6) return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 6, OUT>, batch);
  return cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreadsMany, 8, OUT>, batch);
}

// out_form: kOutNibbles (act_idx = [M][K_pad / 2]) or signed bytes for the tensor-core kernel (act_idx = [M][K_pad],
// kOutBytes in column order, kOutBytes2 in the 2-bit decoder's order).
lcd_status launch_quantize_form(const lcd_act_problem* probs, int count, int out_form, void* stream) {
  QuantProblem all[LCD_MAX_BATCH];
  long long tokens = 0;
  for (int i = 0; i < count; ++i) {
    const lcd_act_problem& a = probs[i];
    QuantProblem& q = all[i];
    q.x = static_cast<const __half*>(a.x_fp16);
    q.inv_smooth = a.inv_smooth;
    q.static_scale = a.static_scale;
    q.act_idx = a.act_idx;
    q.act_scale = a.act_scale;
    q.K = a.K;
    q.K_pad = (long long)round_up_u64((uint64_t)a.K, kTileK);
    q.ldx = a.ldx;
    q.cta0 = (int)a.M;          // (the token count until the launches are formed below)
    q.vec = (reinterpret_cast<uintptr_t>(a.x_fp16) % 16 == 0) && (a.ldx % 8 == 0) && (a.K % 8 == 0) &&
            (a.inv_smooth == nullptr || reinterpret_cast<uintptr_t>(a.inv_smooth) % 16 == 0) &&
            (reinterpret_cast<uintptr_t>(a.act_idx) % (out_form == kOutNibbles ? 4 : 8) == 0);
    tokens += a.M;
    if (tokens > 0x7fffffffLL) return LCD_ERR_INVALID_ARG;
  }
  const bool many = tokens > 296 || out_form != kOutNibbles;      // the byte forms exist for the small CTAs only
  const int threads = many ? kQThreadsMany : kQThreads;
  // register-resident instance a problem's rows fit (0: none, the two-pass instance)
  auto instance_of = [&](const QuantProblem& q) -> int {
    if (!q.vec) return 0;
    const long long chunks = (q.K_pad + 8 * threads - 1) / (8 * threads);
    if (!many) return chunks <= kQChunks ? kQChunks : 0;
    return chunks <= 2 ? 2 : chunks <= 3 ? 3 : chunks <= 4 ? 4 : chunks <= 6 ? 6 : chunks <= 8 ? 8 : 0;
  };
  // Few tokens: one launch, the instance of the longest row.  Many tokens: one launch per instance that occurs, so
  // that short rows are not run through the loops and registers of the longest one.
  bool done[LCD_MAX_BATCH] = {};
  for (int first = 0; first < count; ++first) {
    if (done[first]) continue;
    int inst = instance_of(all[first]);
    QuantBatch batch;
    batch.count = 0;
    long long grid = 0;
    for (int i = first; i < count; ++i) {
      if (done[i]) continue;
      const int mine = instance_of(all[i]);
      if (many && mine != inst) continue;
      if (!many && mine != 0) inst = mine;       // one launch: the kernel itself sends a row that does not fit the two-pass way
      QuantProblem& q = batch.p[batch.count++];
      q = all[i];
      q.cta0 = (int)grid;
      grid += all[i].cta0;
      done[i] = true;
    }
    for (int i = batch.count; i < LCD_MAX_BATCH; ++i) batch.p[i] = batch.p[0];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(threads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (!many)
      e = inst ? cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreads, kQChunks>, batch)
               : cudaLaunchKernelEx(&cfg, smooth_quantize_kernel<kQThreads, 0>, batch);
    else if (out_form == kOutBytes) e = launch_small_ctas<kOutBytes>(cfg, inst, batch);
    else if (out_form == kOutBytes2) e = launch_small_ctas<kOutBytes2>(cfg, inst, batch);
    else e = launch_small_ctas<kOutNibbles>(cfg, inst, batch);
    if (e != cudaSuccess) {
      set_cuda_error((int)e);
      return LCD_ERR_CUDA;
    }
  }
  return LCD_OK;
}

}  // namespace

lcd_status launch_smooth_quantize_batch(const lcd_act_problem* probs, int count, void* stream) {
  return launch_quantize_form(probs, count, kOutNibbles, stream);
}

lcd_status launch_smooth_quantize_dense_levels(const lcd_act_problem* probs, int count, int bits, void* stream) {
  return launch_quantize_form(probs, count, bits == 2 ? kOutBytes2 : kOutBytes, stream);
}

lcd_status launch_smooth_quantize(const void* x, int64_t M, int64_t K, int64_t ldx, const float* inv_smooth,
                                  const float* static_scale, uint8_t* act_idx, float* act_scale, void* stream) {
  lcd_act_problem a;
  a.x_fp16 = x;
  a.M = M;
  a.K = K;
  a.ldx = ldx;
  a.inv_smooth = inv_smooth;
  a.static_scale = static_scale;
  a.act_idx = act_idx;
  a.act_scale = act_scale;
  return launch_smooth_quantize_batch(&a, 1, stream);
}

}  // namespace lcd
