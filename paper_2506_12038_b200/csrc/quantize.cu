// Input transformation (Section 4.1 of the LCD paper): smoothing and uniform symmetric quantisation fused
// into one multiply, round to nearest (ties to even), clip to [-8, 7]; emits 4-bit indices a = q + 8 and
// the per-token scale.  Every operation is a single IEEE binary32 operation in the order stated in
// include/lcd.h, so the indices are reproducible bit for bit.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"

namespace lcd {

constexpr int kQThreads = 512;

__device__ __forceinline__ int quant_level(float v) {
  // round half to even, then clip to the 4-bit symmetric range
  float r = rintf(v);
  r = fminf(fmaxf(r, -8.0f), 7.0f);
  return (int)r;
}

// One CTA per token.  VEC: rows are 16-byte aligned and K is a multiple of 8, so each thread handles 8
// consecutive columns per step (one 16-byte load of x, two of inv_smooth, one 4-byte store).
template <bool VEC>
__global__ void __launch_bounds__(kQThreads)
smooth_quantize_kernel(const __half* __restrict__ x, int64_t K, int64_t K_pad, int64_t ldx,
                       const float* __restrict__ inv_smooth, const float* __restrict__ static_scale,
                       uint8_t* __restrict__ act_idx, float* __restrict__ act_scale) {
  __shared__ float s_red[kQThreads / 32];
  __shared__ float s_mult;
  const int64_t m = blockIdx.x;
  const __half* xr = x + m * ldx;
  uint8_t* out = act_idx + m * (K_pad / 2);
  const int tid = threadIdx.x;
  const bool is_static = static_scale != nullptr;

  if (!is_static) {
    float amax = 0.0f;
    if (VEC) {
      for (int64_t k = (int64_t)tid * 8; k < K; k += (int64_t)kQThreads * 8) {
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
      for (int64_t k = tid; k < K; k += kQThreads) {
        const float f = inv_smooth ? inv_smooth[k] : 1.0f;
        amax = fmaxf(amax, fabsf(__fmul_rn(__half2float(xr[k]), f)));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = amax;
    __syncthreads();
    if (tid < 32) {
      float v = tid < kQThreads / 32 ? s_red[tid] : 0.0f;
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
    for (int64_t k = (int64_t)tid * 8; k < K_pad; k += (int64_t)kQThreads * 8) {
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
          const uint32_t a0 = (uint32_t)(quant_level(t0) + 8), a1 = (uint32_t)(quant_level(t1) + 8);
          packed |= (a0 | (a1 << 4)) << (8 * i);
        }
      }
      *reinterpret_cast<uint32_t*>(out + k / 2) = packed;
    }
  } else {
    for (int64_t j = tid; j < K_pad / 2; j += kQThreads) {
      uint32_t a[2] = {8u, 8u};
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int64_t k = 2 * j + i;
        if (k < K) {
          float t = __fmul_rn(__half2float(xr[k]), inv_smooth ? inv_smooth[k] : 1.0f);
          if (!is_static) t = __fmul_rn(t, r);
          a[i] = (uint32_t)(quant_level(t) + 8);
        }
      }
      out[j] = (uint8_t)(a[0] | (a[1] << 4));
    }
  }
}

lcd_status launch_smooth_quantize(const void* x, int64_t M, int64_t K, int64_t ldx, const float* inv_smooth,
                                  const float* static_scale, uint8_t* act_idx, float* act_scale, void* stream) {
  const int64_t K_pad = (int64_t)round_up_u64((uint64_t)K, kTileK);
  const bool vec = (reinterpret_cast<uintptr_t>(x) % 16 == 0) && (ldx % 8 == 0) && (K % 8 == 0) &&
                   (inv_smooth == nullptr || reinterpret_cast<uintptr_t>(inv_smooth) % 16 == 0) &&
                   (reinterpret_cast<uintptr_t>(act_idx) % 4 == 0);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* xh = static_cast<const __half*>(x);
  if (vec)
    smooth_quantize_kernel<true><<<(unsigned)M, kQThreads, 0, s>>>(xh, K, K_pad, ldx, inv_smooth, static_scale,
                                                                   act_idx, act_scale);
  else
    smooth_quantize_kernel<false><<<(unsigned)M, kQThreads, 0, s>>>(xh, K, K_pad, ldx, inv_smooth, static_scale,
                                                                    act_idx, act_scale);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_cuda_error((int)e);
    return LCD_ERR_CUDA;
  }
  return LCD_OK;
}

}  // namespace lcd
