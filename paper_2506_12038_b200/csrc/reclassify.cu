// Reclassification of weights and centroid offsets (Section 3.2 of the LCD paper), offline bookkeeping after a
// round of weight updates, for per-row codebooks sorted in ascending order:
//   a weight of cluster i with update dw moves to i - 1 when dw < -(C_i - C_{i-1}) / 2, to i + 1 when
//   dw > (C_{i+1} - C_i) / 2 (binary32: one subtraction, one halving; edge clusters have one side);
//   dC_j = sum over the weights that end up in j of (dw + (C_old - C_j)), counts alongside.
// One CTA per row; per-thread compensated sums, combined in binary64 in a fixed order: results are reproducible.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"

namespace lcd {

namespace {

constexpr int kRcThreads = 256;
constexpr int kRcMaxC = 16;

template <int CMAX>
__global__ void __launch_bounds__(kRcThreads) reclassify_kernel(const uint8_t* __restrict__ idx, const uint16_t* __restrict__ codebook,
                                                                const float* __restrict__ delta_w, int64_t K, int64_t ldw, int C,
                                                                uint8_t* __restrict__ new_idx, double* __restrict__ delta_c,
                                                                int32_t* __restrict__ counts, const bool vec) {
  __shared__ float s_c[CMAX];
  __shared__ float s_half[CMAX];            // s_half[i] = (C_{i+1} - C_i) / 2
  __shared__ double s_sum[kRcThreads / 32][CMAX];
  __shared__ int s_cnt[kRcThreads / 32][CMAX];
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < C) s_c[tid] = __half2float(__ushort_as_half(codebook[n * C + tid]));
  __syncthreads();
  if (tid < C - 1) s_half[tid] = __fmul_rn(__fsub_rn(s_c[tid + 1], s_c[tid]), 0.5f);
  __syncthreads();
  // Per thread and cluster: the sum of the arriving updates as an unevaluated pair of binary32 numbers (error-free
  // two-sum: binary64 adds are scarce on this part), and integer counts of members and of arrivals from either side;
  // the centroid differences of the arrivals are added at the end from the counts.
  float hi[CMAX], lo[CMAX];
  int cnt[CMAX], from_left[CMAX], from_right[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) { hi[c] = 0.0f; lo[c] = 0.0f; cnt[c] = 0; from_left[c] = 0; from_right[c] = 0; }
  const uint8_t* ir = idx + n * K;
  const float* dr = delta_w + n * ldw;
  uint8_t* outr = new_idx + n * K;
  auto one = [&](int i, float dw) {
    int j = i;
    if (i > 0 && dw < -s_half[i - 1]) j = i - 1;
    else if (i < C - 1 && dw > s_half[i]) j = i + 1;
#pragma unroll
    for (int c = 0; c < CMAX; ++c) {
      const bool mine = c == j;
      const float x = mine ? dw : 0.0f;
      const float t = __fadd_rn(hi[c], x);                       // two-sum of (hi, x)
      const float bb = __fsub_rn(t, hi[c]);
      const float err = __fadd_rn(__fsub_rn(hi[c], __fsub_rn(t, bb)), __fsub_rn(x, bb));
      hi[c] = t;
      lo[c] = __fadd_rn(lo[c], err);
      cnt[c] += mine ? 1 : 0;
      from_left[c] += (mine && i < j) ? 1 : 0;
      from_right[c] += (mine && i > j) ? 1 : 0;
    }
    return (uint32_t)j;
  };
  if (vec) {      // 16 weights per thread and step: one 16-byte index load, four 16-byte update loads, one 16-byte store
    for (int64_t k = (int64_t)tid * 16; k < K; k += (int64_t)kRcThreads * 16) {
      const uint4 iv = __ldg(reinterpret_cast<const uint4*>(ir + k));
      const uint32_t iw[4] = {iv.x, iv.y, iv.z, iv.w};
      uint32_t ow[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 d = __ldg(reinterpret_cast<const float4*>(dr + k + 4 * q));
        const float dv[4] = {d.x, d.y, d.z, d.w};
        uint32_t o = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) o |= one((int)((iw[q] >> (8 * e)) & 0xffu), dv[e]) << (8 * e);
        ow[q] = o;
      }
      *reinterpret_cast<uint4*>(outr + k) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
    }
  } else {
    for (int64_t k = tid; k < K; k += kRcThreads) outr[k] = (uint8_t)one(ir[k], dr[k]);
  }
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    double v = (double)hi[c] + (double)lo[c];
    if (c < C) {
      if (c > 0) v += (double)from_left[c] * ((double)s_c[c - 1] - (double)s_c[c]);
      if (c < C - 1) v += (double)from_right[c] * ((double)s_c[c + 1] - (double)s_c[c]);
    }
    int q = cnt[c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      v += __shfl_xor_sync(0xffffffffu, v, o);
      q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (lane == 0) { s_sum[warp][c] = v; s_cnt[warp][c] = q; }
  }
  __syncthreads();
  if (tid < C) {
    double v = 0.0;
    int q = 0;
    for (int w = 0; w < kRcThreads / 32; ++w) { v += s_sum[w][tid]; q += s_cnt[w][tid]; }
    delta_c[n * C + tid] = v;
    counts[n * C + tid] = q;
  }
}

}  // namespace

lcd_status launch_reclassify(const uint8_t* idx, const uint16_t* codebook, const float* delta_w, int64_t N, int64_t K,
                             int64_t ldw, int C, uint8_t* new_idx, double* delta_c, int32_t* counts, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  const bool vec = K % 16 == 0 && ldw % 4 == 0 && al16(idx) && al16(delta_w) && al16(new_idx);
  if (C <= 4) reclassify_kernel<4><<<(unsigned)N, kRcThreads, 0, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  else if (C <= 8) reclassify_kernel<8><<<(unsigned)N, kRcThreads, 0, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  else reclassify_kernel<kRcMaxC><<<(unsigned)N, kRcThreads, 0, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
