// Adaptive smoothing search (Section 3.4 of the LCD paper), offline: for every candidate migration strength alpha
// the per-channel factors s_k = xmax_k^alpha / wmax_k^(1 - alpha) and the objective
// MSE(X, Q_INT8(X / s) * s) over a calibration batch; the candidate with the smallest error wins and its 1/s_k
// are written for the online input transformation.  The level decisions use the binary32 steps of the 8-bit
// quantiser (quantize8.cu); reconstruction and sums are binary64 in a fixed order, so results are reproducible.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"

namespace lcd {

namespace {

constexpr int kMaxAlphas = 64;
struct AlphaList {
  int count;
  float a[kMaxAlphas];
};

// xmax[k] = max over the batch of |x[t][k]|
__global__ void __launch_bounds__(256) column_absmax_kernel(const __half* __restrict__ x, int64_t T, int64_t K, int64_t ldx,
                                                            float* __restrict__ xmax) {
  const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (k >= K) return;
  float m = 0.0f;
  for (int64_t t = 0; t < T; ++t) m = fmaxf(m, fabsf(__half2float(x[t * ldx + k])));
  xmax[k] = m;
}

// s[g][k]: binary64 powers, one rounding to binary32; zero maxima leave the channel alone; clamp to [1e-5, 1e5]
__global__ void __launch_bounds__(256) smoothing_factors_kernel(const float* __restrict__ xmax, const float* __restrict__ wmax,
                                                                int64_t K, const AlphaList alphas, float* __restrict__ s) {
  const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int g = blockIdx.y;
  if (k >= K) return;
  const double xm = (double)xmax[k], wm = (double)wmax[k], al = (double)alphas.a[g];
  double v = 1.0;
  if (xm > 0.0 && wm > 0.0) v = pow(xm, al) / pow(wm, 1.0 - al);
  v = fmin(fmax(v, 1e-5), 1e5);
  s[(int64_t)g * K + k] = (float)v;
}

// partial[g][t] = sum_k (x - level * s_q * s)^2 of token t under candidate g
__global__ void __launch_bounds__(256) smoothing_error_kernel(const __half* __restrict__ x, int64_t K, int64_t ldx,
                                                              const float* __restrict__ s, double* __restrict__ partial,
                                                              int64_t T) {
  __shared__ float s_f[8];
  __shared__ double s_d[8];
  __shared__ float s_amax;
  const int64_t t = blockIdx.x;
  const int g = blockIdx.y;
  const __half* xr = x + t * ldx;
  const float* sg = s + (int64_t)g * K;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float amax = 0.0f;
  for (int64_t k = tid; k < K; k += 256)
    amax = fmaxf(amax, fabsf(__fmul_rn(__half2float(xr[k]), __fdiv_rn(1.0f, sg[k]))));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) s_f[warp] = amax;
  __syncthreads();
  if (tid == 0) {
    float v = 0.0f;
    for (int w = 0; w < 8; ++w) v = fmaxf(v, s_f[w]);
    s_amax = v;
  }
  __syncthreads();
  const float A = s_amax;
  const float r = A > 0.0f ? __fdiv_rn(127.0f, A) : 0.0f;
  const double sq = A > 0.0f ? (double)__fdiv_rn(A, 127.0f) : 1.0;
  double err = 0.0;
  for (int64_t k = tid; k < K; k += 256) {
    const float xv = __half2float(xr[k]);
    const float sk = sg[k];
    float lev = rintf(__fmul_rn(__fmul_rn(xv, __fdiv_rn(1.0f, sk)), r));
    lev = fminf(fmaxf(lev, -128.0f), 127.0f);
    const double d = (double)xv - (double)lev * sq * (double)sk;
    err += d * d;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
  if (lane == 0) s_d[warp] = err;
  __syncthreads();
  if (tid == 0) {
    double v = 0.0;
    for (int w = 0; w < 8; ++w) v += s_d[w];
    partial[(int64_t)g * T + t] = v;
  }
}

// mse[g] = sum_t partial[g][t] / (T * K) in token order; best = first smallest; inv_smooth = 1 / s[best]
__global__ void __launch_bounds__(256) smoothing_pick_kernel(const double* __restrict__ partial, int64_t T, int64_t K, int G,
                                                             const float* __restrict__ s, double* __restrict__ mse,
                                                             int32_t* __restrict__ best, float* __restrict__ inv_smooth) {
  __shared__ double s_mse[kMaxAlphas];
  __shared__ int s_best;
  const int tid = threadIdx.x;
  if (tid < G) {
    double v = 0.0;
    for (int64_t t = 0; t < T; ++t) v += partial[(int64_t)tid * T + t];
    v /= (double)T * (double)K;
    s_mse[tid] = v;
    mse[tid] = v;
  }
  __syncthreads();
  if (tid == 0) {
    int b = 0;
    for (int g = 1; g < G; ++g)
      if (s_mse[g] < s_mse[b]) b = g;
    s_best = b;
    if (best) *best = b;
  }
  __syncthreads();
  if (inv_smooth)
    for (int64_t k = tid; k < K; k += 256) inv_smooth[k] = __fdiv_rn(1.0f, s[(int64_t)s_best * K + k]);
}

size_t align256s(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

size_t smoothing_search_workspace_bytes(int64_t T, int64_t K, int G) {
  return align256s((size_t)K * sizeof(float)) + align256s((size_t)G * K * sizeof(float)) + align256s((size_t)G * T * sizeof(double));
}

lcd_status launch_smoothing_search(const void* x, int64_t T, int64_t K, int64_t ldx, const float* wmax, const float* alphas_host,
                                   int G, void* workspace, double* mse, int32_t* best, float* inv_smooth, void* stream) {
  AlphaList al;
  al.count = G;
  for (int i = 0; i < kMaxAlphas; ++i) al.a[i] = i < G ? alphas_host[i] : 0.0f;
  uint8_t* base = static_cast<uint8_t*>(workspace);
  float* xmax = reinterpret_cast<float*>(base);
  float* s = reinterpret_cast<float*>(base + align256s((size_t)K * sizeof(float)));
  double* partial = reinterpret_cast<double*>(base + align256s((size_t)K * sizeof(float)) + align256s((size_t)G * K * sizeof(float)));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __half* xh = static_cast<const __half*>(x);
  const unsigned kb = (unsigned)((K + 255) / 256);
  column_absmax_kernel<<<kb, 256, 0, st>>>(xh, T, K, ldx, xmax);
  smoothing_factors_kernel<<<dim3(kb, (unsigned)G), 256, 0, st>>>(xmax, wmax, K, al, s);
  smoothing_error_kernel<<<dim3((unsigned)T, (unsigned)G), 256, 0, st>>>(xh, K, ldx, s, partial, T);
  smoothing_pick_kernel<<<1, 256, 0, st>>>(partial, T, K, G, s, mse, best, inv_smooth);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
