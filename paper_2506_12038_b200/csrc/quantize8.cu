// Input transformation with 8-bit levels (Section 4.1 of the LCD paper with its own b = 8): the steps of
// quantize.cu with 127 in place of 7, clip to [-128, 127], one signed byte per column.  Every operation is a
// single IEEE binary32 operation in the order stated in include/lcd.h.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"

namespace lcd {

namespace {

// The signed byte of round-half-to-even(v) clipped to [-128, 127].  Clipping first gives the same level (integer
// bounds); adding 1.5 * 2^23 rounds to an integer, ties to even, in one binary32 addition and leaves the level's
// two's complement in the low byte of the sum.
__device__ __forceinline__ uint32_t level8(float v) {
  const float u = fminf(fmaxf(v, -128.0f), 127.0f);
  return __float_as_uint(__fadd_rn(u, 12582912.0f)) & 0xffu;
}

// One token per CTA.  vec: rows are 16-byte aligned and K is a multiple of 8: 8 columns per thread and step.
template <int THREADS>
__device__ __forceinline__ void quantize8_token(const __half* __restrict__ x, int64_t m, int64_t K, int64_t K_pad,
                                                int64_t ldx, const float* __restrict__ inv_smooth,
                                                const float* __restrict__ static_scale, int8_t* __restrict__ act_q,
                                                float* __restrict__ act_scale, const bool VEC) {
  __shared__ float s_red[THREADS / 32];
  __shared__ float s_mult;
  const __half* xr = x + m * ldx;
  int8_t* out = act_q + m * K_pad;
  const int tid = threadIdx.x;
  const bool is_static = static_scale != nullptr;
  auto load8 = [&](int64_t k, float (&t)[8]) {     // t = x * inv_smooth for columns k .. k + 7
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
      t[2 * i] = __fmul_rn(v.x, f[2 * i]);
      t[2 * i + 1] = __fmul_rn(v.y, f[2 * i + 1]);
    }
  };

  if (!is_static) {
    float amax = 0.0f;
    if (VEC) {
      for (int64_t k = (int64_t)tid * 8; k < K; k += (int64_t)THREADS * 8) {
        float t[8];
        load8(k, t);
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(t[i]));
      }
    } else {
      for (int64_t k = tid; k < K; k += THREADS)
        amax = fmaxf(amax, fabsf(__fmul_rn(__half2float(xr[k]), inv_smooth ? inv_smooth[k] : 1.0f)));
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
          sq = __fdiv_rn(v, 127.0f);
          r = __fdiv_rn(127.0f, v);
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
      uint2 packed = make_uint2(0u, 0u);           // padding columns are level 0
      if (k < K) {
        float t[8];
        load8(k, t);
        uint32_t b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) b[i] = level8(is_static ? t[i] : __fmul_rn(t[i], r));
        packed.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
        packed.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
      }
      *reinterpret_cast<uint2*>(out + k) = packed;
    }
  } else {
    for (int64_t k = tid; k < K_pad; k += THREADS) {
      uint32_t b = 0;
      if (k < K) {
        const float t = __fmul_rn(__half2float(xr[k]), inv_smooth ? inv_smooth[k] : 1.0f);
        b = level8(is_static ? t : __fmul_rn(t, r));
      }
      out[k] = (int8_t)b;
    }
  }
}


struct Quant8Problem {
  const __half* x;
  const float* inv_smooth;
  const float* static_scale;
  int8_t* act_q;
  float* act_scale;
  long long K, K_pad, ldx;
  int vec;
  int token0;      // first CTA of this problem
};
struct Quant8Batch {
  int count;
  Quant8Problem p[LCD_MAX_BATCH];
};

template <int THREADS>
__global__ void __launch_bounds__(THREADS) smooth_quantize8_kernel(const Quant8Batch B) {
  int pi = 0;
  for (int i = 1; i < B.count; ++i)
    if ((int)blockIdx.x >= B.p[i].token0) pi = i;
  const Quant8Problem& P = B.p[pi];
  asm volatile("griddepcontrol.wait;" ::: "memory");           // x may be written by the previous kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  quantize8_token<THREADS>(P.x, (int64_t)blockIdx.x - P.token0, P.K, P.K_pad, P.ldx, P.inv_smooth, P.static_scale,
                           P.act_q, P.act_scale, P.vec != 0);
}

bool fill_quant8(Quant8Problem& q, const void* x, int64_t K, int64_t ldx, const float* inv_smooth,
                 const float* static_scale, int8_t* act_q, float* act_scale) {
  q.x = static_cast<const __half*>(x);
  q.inv_smooth = inv_smooth;
  q.static_scale = static_scale;
  q.act_q = act_q;
  q.act_scale = act_scale;
  q.K = K;
  q.K_pad = (long long)round_up_u64((uint64_t)K, kTileK);
  q.ldx = ldx;
  q.vec = (K % 8 == 0) && (ldx % 8 == 0) && ((reinterpret_cast<uintptr_t>(x) & 15) == 0) &&
          (!inv_smooth || (reinterpret_cast<uintptr_t>(inv_smooth) & 15) == 0) &&
          ((reinterpret_cast<uintptr_t>(act_q) & 7) == 0);
  return true;
}

lcd_status launch_quant8(const Quant8Batch& batch, int64_t tokens, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)tokens);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (tokens > 296) {       // many tokens: small CTAs, several per SM
    cfg.blockDim = dim3(256);
    e = cudaLaunchKernelEx(&cfg, smooth_quantize8_kernel<256>, batch);
  } else {
    cfg.blockDim = dim3(1024);
    e = cudaLaunchKernelEx(&cfg, smooth_quantize8_kernel<1024>, batch);
  }
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace

lcd_status launch_smooth_quantize8(const void* x, int64_t M, int64_t K, int64_t ldx, const float* inv_smooth,
                                   const float* static_scale, int8_t* act_q, float* act_scale, void* stream) {
  Quant8Batch batch;
  batch.count = 1;
  fill_quant8(batch.p[0], x, K, ldx, inv_smooth, static_scale, act_q, act_scale);
  batch.p[0].token0 = 0;
  for (int i = 1; i < LCD_MAX_BATCH; ++i) batch.p[i] = batch.p[0];
  return launch_quant8(batch, M, static_cast<cudaStream_t>(stream));
}

lcd_status launch_smooth_quantize8_batch(const lcd_act_problem* probs, int count, void* stream) {
  Quant8Batch batch;
  batch.count = count;
  int64_t tokens = 0;
  for (int i = 0; i < count; ++i) {
    fill_quant8(batch.p[i], probs[i].x_fp16, probs[i].K, probs[i].ldx, probs[i].inv_smooth, probs[i].static_scale,
                reinterpret_cast<int8_t*>(probs[i].act_idx), probs[i].act_scale);
    batch.p[i].token0 = (int)tokens;
    tokens += probs[i].M;
    if (tokens > 0x7fffffffLL) return LCD_ERR_INVALID_ARG;
  }
  for (int i = count; i < LCD_MAX_BATCH; ++i) batch.p[i] = batch.p[0];
  return launch_quant8(batch, tokens, static_cast<cudaStream_t>(stream));
}

}  // namespace lcd
