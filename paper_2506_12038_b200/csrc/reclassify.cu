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
  __shared__ float s_gl[CMAX], s_gr[CMAX];  // half-gaps (C_i - C_{i-1}) / 2 and (C_{i+1} - C_i) / 2, infinite at the edges
  __shared__ float s_wh[kRcThreads / 32][CMAX], s_wl[kRcThreads / 32][CMAX];
  __shared__ int s_cnt[kRcThreads / 32][CMAX], s_wfl[kRcThreads / 32][CMAX], s_wfr[kRcThreads / 32][CMAX];
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < C) s_c[tid] = __half2float(__ushort_as_half(codebook[n * C + tid]));
  __syncthreads();
  if (tid < CMAX) {
    const float inf = __int_as_float(0x7f800000);
    s_gl[tid] = (tid > 0 && tid < C) ? __fmul_rn(__fsub_rn(s_c[tid], s_c[tid - 1]), 0.5f) : inf;
    s_gr[tid] = (tid < C - 1) ? __fmul_rn(__fsub_rn(s_c[tid + 1], s_c[tid]), 0.5f) : inf;
  }
  __syncthreads();
  // Per thread and cluster, in the thread's own column of shared memory (indexed by the data-dependent cluster; a
  // register array would need one predicated copy of every operation per cluster): the sum of the arriving updates
  // as an unevaluated pair of binary32 numbers (error-free two-sum: binary64 adds are scarce on this part) and
  // integer counts of members and of arrivals from either side; the centroid differences of the arrivals are
  // added at the end from the counts.
  extern __shared__ unsigned long long s_dyn[];
  float2* s_pair = reinterpret_cast<float2*>(s_dyn);                      // [CMAX][kRcThreads] (hi, lo)
  unsigned long long* s_cnt3 = s_dyn + CMAX * kRcThreads;                 // members | arrivals from the left << 21
                                                                          // | arrivals from the right << 42
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    s_pair[c * kRcThreads + tid] = make_float2(0.0f, 0.0f);
    s_cnt3[c * kRcThreads + tid] = 0ull;
  }
  const uint8_t* ir = idx + n * K;
  const float* dr = delta_w + n * ldw;
  uint8_t* outr = new_idx + n * K;
  // branch-free: s_gl[i] / s_gr[i] are the half-gaps to the left / right of cluster i, infinite at the edges
  auto one = [&](int i, float dw) {
    const int left = dw < -s_gl[i] ? 1 : 0;
    const int right = (dw > s_gr[i] ? 1 : 0) & (left ^ 1);
    const int j = i - left + right;
    const int slot = j * kRcThreads + tid;
    const float2 p = s_pair[slot];
    const float t = __fadd_rn(p.x, dw);                          // two-sum of (hi, dw)
    const float bb = __fsub_rn(t, p.x);
    const float err = __fadd_rn(__fsub_rn(p.x, __fsub_rn(t, bb)), __fsub_rn(dw, bb));
    s_pair[slot] = make_float2(t, __fadd_rn(p.y, err));
    s_cnt3[slot] += 1ull + ((unsigned long long)right << 21) + ((unsigned long long)left << 42);
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
  // Block reduction of the pairs and counts, still in binary32 pairs (binary64 operations only on the C final values
  // of the row: they are slow enough here that a few dozen per thread dominated the kernel), fixed order.
  auto two_sum = [](float& h, float& l, float h2, float l2) {
    const float t = __fadd_rn(h, h2);
    const float bb = __fsub_rn(t, h);
    const float err = __fadd_rn(__fsub_rn(h, __fsub_rn(t, bb)), __fsub_rn(h2, bb));
    h = t;
    l = __fadd_rn(__fadd_rn(l, l2), err);
  };
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    const int slot = c * kRcThreads + tid;
    float h = s_pair[slot].x, l = s_pair[slot].y;
    const unsigned long long c3 = s_cnt3[slot];
    int q = (int)(c3 & 0x1fffffull), fl = (int)((c3 >> 21) & 0x1fffffull), fr = (int)((c3 >> 42) & 0x1fffffull);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float h2 = __shfl_xor_sync(0xffffffffu, h, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
      two_sum(h, l, h2, l2);
      q += __shfl_xor_sync(0xffffffffu, q, o);
      fl += __shfl_xor_sync(0xffffffffu, fl, o);
      fr += __shfl_xor_sync(0xffffffffu, fr, o);
    }
    if (lane == 0) {
      s_wh[warp][c] = h; s_wl[warp][c] = l; s_cnt[warp][c] = q; s_wfl[warp][c] = fl; s_wfr[warp][c] = fr;
    }
  }
  __syncthreads();
  if (tid < C) {
    float h = 0.0f, l = 0.0f;
    int q = 0, fl = 0, fr = 0;
    for (int w = 0; w < kRcThreads / 32; ++w) {
      two_sum(h, l, s_wh[w][tid], s_wl[w][tid]);
      q += s_cnt[w][tid]; fl += s_wfl[w][tid]; fr += s_wfr[w][tid];
    }
    double v = (double)h + (double)l;
    if (tid > 0) v += (double)fl * ((double)s_c[tid - 1] - (double)s_c[tid]);
    if (tid < C - 1) v += (double)fr * ((double)s_c[tid + 1] - (double)s_c[tid]);
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
  if (C <= 4) reclassify_kernel<4><<<(unsigned)N, kRcThreads, 4 * kRcThreads * 16, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  else if (C <= 8) reclassify_kernel<8><<<(unsigned)N, kRcThreads, 8 * kRcThreads * 16, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  else {
    static bool attr_set = false;     // 80 KB of dynamic shared memory needs the opt-in
    if (!attr_set) {
      const cudaError_t ea = cudaFuncSetAttribute(reclassify_kernel<kRcMaxC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  kRcMaxC * kRcThreads * 16);
      if (ea != cudaSuccess) { set_cuda_error((int)ea); return LCD_ERR_CUDA; }
      attr_set = true;
    }
    reclassify_kernel<kRcMaxC><<<(unsigned)N, kRcThreads, kRcMaxC * kRcThreads * 16, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
