// Reclassification of weights and centroid offsets (Section 3.2 of the LCD paper), offline bookkeeping after a
// round of weight updates, for per-row codebooks sorted in ascending order:
//   a weight of cluster i with update dw moves to i - 1 when dw < -(C_i - C_{i-1}) / 2, to i + 1 when
//   dw > (C_{i+1} - C_i) / 2 (binary32: one subtraction, one halving; edge clusters have one side);
//   dC_j = sum over the weights that end up in j of (dw + (C_old - C_j)), counts alongside.
// One CTA per row; per-thread compensated sums, combined in binary64 in a fixed order: results are reproducible.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "device_util.h"

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
  __shared__ float2 s_gap[CMAX];            // half-gaps (C_i - C_{i-1}) / 2 and (C_{i+1} - C_i) / 2, infinite at the edges
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < C) s_c[tid] = __half2float(__ushort_as_half(codebook[n * C + tid]));
  __syncthreads();
  if (tid < CMAX) {
    const float inf = __int_as_float(0x7f800000);
    s_gap[tid] = make_float2((tid > 0 && tid < C) ? __fmul_rn(__fsub_rn(s_c[tid], s_c[tid - 1]), 0.5f) : inf,
                             (tid < C - 1) ? __fmul_rn(__fsub_rn(s_c[tid + 1], s_c[tid]), 0.5f) : inf);
  }
  __syncthreads();
  // Per thread and cluster, in the thread's own column of shared memory (indexed by the data-dependent cluster; a
  // register array would need one predicated copy of every operation per cluster): the sum of the arriving updates
  // as an unevaluated pair of binary32 numbers (error-free two-sum: binary64 adds are scarce on this part) and
  // integer counts of members and of arrivals from either side; the centroid differences of the arrivals are
  // added at the end from the counts.
  extern __shared__ uint4 s_dyn[];
  // one 16-byte slot per thread and cluster: (hi, lo, counts low word, counts high word); the 64-bit count word is
  // members | arrivals from the left << 21 | arrivals from the right << 42.  One load and one store per weight: the
  // load/store unit's queue is what bounds this kernel.
  uint4* s_slot = s_dyn;                                                  // [CMAX][kRcThreads]
#pragma unroll
  for (int c = 0; c < CMAX; ++c) s_slot[c * kRcThreads + tid] = make_uint4(0u, 0u, 0u, 0u);
  const uint8_t* ir = idx + n * K;
  const float* dr = delta_w + n * ldw;
  uint8_t* outr = new_idx + n * K;
  // branch-free: s_gap[i] = (half-gap to the left, half-gap to the right) of cluster i, infinite at the edges.
  // An index is reduced to the table size CMAX before it addresses shared memory, so a byte >= C (the caller's
  // error) cannot reach outside the slots: such a weight keeps its reduced index and is counted in no cluster.
  auto one = [&](int i, float dw) {
    const float2 gap = s_gap[i];
    const int left = dw < -gap.x ? 1 : 0;
    const int right = (dw > gap.y ? 1 : 0) & (left ^ 1);
    const int j = i - left + right;
    const int slot = j * kRcThreads + tid;
    uint4 v = s_slot[slot];
    const float h = __uint_as_float(v.x), l = __uint_as_float(v.y);
    const float t = __fadd_rn(h, dw);                            // two-sum of (hi, dw)
    const float bb = __fsub_rn(t, h);
    const float err = __fadd_rn(__fsub_rn(h, __fsub_rn(t, bb)), __fsub_rn(dw, bb));
    unsigned long long cnt = ((unsigned long long)v.w << 32) | v.z;
    cnt += 1ull + ((unsigned long long)right << 21) + ((unsigned long long)left << 42);
    v.x = __float_as_uint(t);
    v.y = __float_as_uint(__fadd_rn(l, err));
    v.z = (uint32_t)cnt;
    v.w = (uint32_t)(cnt >> 32);
    s_slot[slot] = v;
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
        for (int e = 0; e < 4; ++e) o |= one((int)((iw[q] >> (8 * e)) & (uint32_t)(CMAX - 1)), dv[e]) << (8 * e);
        ow[q] = o;
      }
      *reinterpret_cast<uint4*>(outr + k) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
    }
  } else {
    for (int64_t k = tid; k < K; k += kRcThreads) outr[k] = (uint8_t)one(ir[k] & (CMAX - 1), dr[k]);
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
  // One warp folds the 256 columns of slots: every lane adds its eight columns, then a butterfly over the lanes.
  // (A butterfly in every warp made this reduction as expensive as the 16 weights a thread handles per 4096 columns.)
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int c = 0; c < CMAX; ++c) {
      float h = 0.0f, l = 0.0f;
      unsigned long long c3 = 0ull;
#pragma unroll
      for (int w = 0; w < kRcThreads / 32; ++w) {
        const uint4 sv = s_slot[c * kRcThreads + w * 32 + lane];
        two_sum(h, l, __uint_as_float(sv.x), __uint_as_float(sv.y));
        c3 += ((unsigned long long)sv.w << 32) | sv.z;          // K <= 2^25: a thread counts at most 2^17, eight of them 2^20 < 2^21
      }
      // fields of the packed count word may carry into each other once summed over threads: unpack before the lanes meet
      int q = (int)(c3 & 0x1fffffull), fl = (int)((c3 >> 21) & 0x1fffffull), fr = (int)((c3 >> 42) & 0x1fffffull);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float h2 = __shfl_xor_sync(0xffffffffu, h, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
        two_sum(h, l, h2, l2);
        q += __shfl_xor_sync(0xffffffffu, q, o);
        fl += __shfl_xor_sync(0xffffffffu, fl, o);
        fr += __shfl_xor_sync(0xffffffffu, fr, o);
      }
      if (lane == 0 && c < C) {
        double v = (double)h + (double)l;
        if (c > 0) v += (double)fl * ((double)s_c[c - 1] - (double)s_c[c]);
        if (c < C - 1) v += (double)fr * ((double)s_c[c + 1] - (double)s_c[c]);
        delta_c[n * C + c] = v;
        counts[n * C + c] = q;
      }
    }
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
    static PerDeviceFlag attr_set;    // 80 KB of dynamic shared memory needs the opt-in, on every device
    int dev;
    if (attr_set.first(&dev)) {
      const cudaError_t ea = cudaFuncSetAttribute(reclassify_kernel<kRcMaxC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  kRcMaxC * kRcThreads * 16);
      if (ea != cudaSuccess) { set_cuda_error((int)ea); return LCD_ERR_CUDA; }
      attr_set.done(dev);
    }
    reclassify_kernel<kRcMaxC><<<(unsigned)N, kRcThreads, kRcMaxC * kRcThreads * 16, s>>>(idx, codebook, delta_w, K, ldw, C, new_idx, delta_c, counts, vec);
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
