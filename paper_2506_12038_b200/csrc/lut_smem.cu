// LUT-GEMV for ONE token and 2-bit weight indices with the bucket tables of Section 4.2 of the LCD paper
// (centroid-stationary buckets: per output row and centroid w the sum S_w of the activation levels whose weight
// index is w, then y = s_q * sum_w cb[w] * S_w) held in shared memory.
//
// Table.  A byte of the index area holds the indices of four consecutive columns of one row.  For every such
// group of four columns the CTA builds a 256-entry table indexed by that byte; an entry is one 32-bit word whose
// byte w is the partial bucket sum of those four columns for centroid w (levels a = q + 8, a column that does not
// fall into bucket w adds 8, so every byte is S_w + 32 and fits 8 unsigned bits).  One shared-memory load looks
// four weights up for all four buckets.  A table costs 1 KB per four columns, so a CTA works on a slice of at most
// W blocks of 256 columns (W x 64 KB) and on many rows of it.
//
// Banks.  The table of group G of a block lives in one bank: word address = entry * 64 + 32 * ((G >> 2) & 1) +
// 16 * (G >> 5) + 4 * ((G >> 3) & 3) + (G & 3).  Lane l = 4g + t of a warp owns 16 bytes of row g of a tile, the
// byte groups {32h + 8t + p}; the lanes take their bytes in an order that depends on g (k-block h = g >> 2 first,
// byte (s + g) & 3 of a word at step s), so the 32 lanes of every lookup hit 32 different banks.  The address is
// formed by one PRMT: byte 0 = the lane's bank offset for the step (a register of four constants), byte 1 = the
// index byte, bytes 2..3 = 0; block and half-row offsets are immediates, which requires the tables to start at a
// fixed address of the shared-memory window (kTableAddr).
//
// Accumulation.  The looked-up words are the A fragments of m16n8k32 u8 x s8 MMAs against a constant 0/1 matrix
// that routes byte w of every word to output column w: one instruction widens the four byte fields to int32, adds
// them over the four lanes (quarters) of a row and over two words, for 16 rows.  Exact integers.
//
// Decomposition.  The work of a launch is the sequence (problem, column slice, 16-row group); it is cut into one
// contiguous piece per CTA (the cut counts the table build of every slice a piece touches).  Each of a CTA's 16
// warps takes every 16th row group of a piece and streams its index bytes through its own ring of bulk copies.
// Per slice a row's four bucket sums are added to zero-filled scratch [row][4] as fp32 (integers below 2^24, so
// the additions are exact and their order does not matter: one vector reduction per row).  When every CTA of the
// launch has added its last sum (a counter in the scratch that all CTAs wait for, bounded; the launch is
// cooperative, so all of them are resident), the rows of all problems are dealt to all threads of the grid: each
// takes a row's totals back, leaves zeros, forms s_q * sum_w cb[w] * S_w and writes y.  Results are bit-identical
// from run to run.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "device_util.h"

namespace lcd {

namespace {

constexpr int kMaxSmem = 227 * 1024;
constexpr uint32_t kBlockBytes = 0x10000u;  // tables of one 256-column block: 64 groups x 256 entries x 4 bytes
constexpr int kItemBytes = 1024;            // one 16-row x 256-column item at 2 bit
constexpr int kMiscBytes = 512;             // mbarriers, partial maxima
constexpr int kMaxCta = 304;
constexpr unsigned long long kTimeoutNs = 2000000000ull;

// Shape of one kernel instance: W table blocks per slice, DEPTH ring slots per warp, WARPS warps per CTA.
// Shared memory: [window start, +kMiscBytes) barriers and maxima | ring | (gap) | tables at the FIXED window address
// kTableAddr (the lookups carry it as an immediate).  The window of a CTA's dynamic shared memory starts 1 KB into
// the shared window on this architecture; the kernel checks what it finds and gives up cleanly otherwise.
template <int W, int DEPTH, int WARPS>
struct Shape {
  static constexpr int kThreads = WARPS * 32;
  static constexpr uint32_t kSlot = W * kItemBytes;
  static constexpr uint32_t kRingBytes = WARPS * DEPTH * kSlot;
  static constexpr uint32_t kTableAddr = (0x400u + kMiscBytes + kRingBytes + 0x3ffu) & ~0x3ffu;
  static constexpr uint32_t kSmemBytes = kTableAddr + W * kBlockBytes;      // dynamic bytes asked for
  static_assert(kSmemBytes <= (uint32_t)kMaxSmem, "tables and ring exceed the shared memory of a CTA");
};

struct SbProblem {
  const uint8_t* items;
  const uint16_t* codebook;
  const uint8_t* act_idx;
  const float* act_scale;
  const __half* x;
  const float* inv_smooth;
  float* y;
  float* sums;        // scratch [N_pad][4] fp32 bucket sums, zero on entry and on exit
  int K, N, N_pad, n_rp, n_kt, n_slices, act_bits, x_vec;
};

struct SbBatch {
  int count, n_cta;
  float* sq;          // scratch [LCD_MAX_BATCH]: s_q of the fused problems, zero on entry and on exit
  int* gate;          // scratch [2]: CTAs that have added all their sums / that have written their rows; zero on entry and exit
  int row0[LCD_MAX_BATCH + 1];   // first row of every problem in the launch-wide row numbering (N_pad rows each)
  SbProblem p[LCD_MAX_BATCH];
  uint2 start[kMaxCta + 1];   // x = problem << 16 | slice, y = row group; entry n_cta is the end
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// D += A * B for the 0/1 routing matrix: byte w of every A word goes to output column w
__device__ __forceinline__ void mma_u8(int& d0, int& d1, int& d2, int& d3, uint32_t a0, uint32_t a1, uint32_t a2,
                                       uint32_t a3, uint32_t b) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%8}, {%0,%1,%2,%3};"
      : "+r"(d0), "+r"(d1), "+r"(d2), "+r"(d3)
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b));
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 1023u) == 0 && globaltimer() - t0 > kTimeoutNs) return false;
  }
}
// One lookup: the table word of index byte ((s + g) & 3) of `w`; IMM = table address, block and half-row offset.
template <uint32_t IMM>
__device__ __forceinline__ uint32_t lookup(uint32_t w, uint32_t c, uint32_t sel) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(prmt(w, c, sel)), "n"(IMM));
  return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void red_add_v4(float* dst, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(dst), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Column slice s of a problem: item columns [kt0, kt0 + width).
__device__ __forceinline__ void slice_range(const SbProblem& P, int s, int* kt0, int* width) {
  const int a = s * P.n_kt / P.n_slices, b = (s + 1) * P.n_kt / P.n_slices;
  *kt0 = a;
  *width = b - a;
}

// The CTA's piece [start, end) of the sequence (problem, slice, row group).
struct Piece {
  const SbBatch& B;
  int end_p, end_s, end_rp;
  __device__ __forceinline__ int seg_end(int p, int s) const {
    return (p == end_p && s == end_s) ? end_rp : B.p[p].n_rp;
  }
  __device__ __forceinline__ bool at_end(int p, int s, int rp) const {
    return p > end_p || (p == end_p && (s > end_s || (s == end_s && rp >= end_rp)));
  }
  // moves (p, s) to the next segment; false when the piece is exhausted
  __device__ __forceinline__ bool next_segment(int& p, int& s) const {
    if (++s == B.p[p].n_slices) { s = 0; ++p; }
    return !at_end(p, s, 0);
  }
};

// All lookups and MMAs of one 8-byte half (k-block) of a lane's two 16-byte records: words (x0, y0) of the tile of
// rows g, (x1, y1) of the tile of rows g + 8.  IMM: table address + block offset.
template <uint32_t IMM>
__device__ __forceinline__ void half_item(uint32_t x0, uint32_t y0, uint32_t x1, uint32_t y1, uint32_t c,
                                          const uint32_t (&sel)[4], uint32_t bsel, int (&a)[4], int (&b)[4]) {
  mma_u8(a[0], a[1], a[2], a[3], lookup<IMM>(x0, c, sel[0]), lookup<IMM>(x1, c, sel[0]), lookup<IMM>(x0, c, sel[1]),
         lookup<IMM>(x1, c, sel[1]), bsel);
  mma_u8(b[0], b[1], b[2], b[3], lookup<IMM>(x0, c, sel[2]), lookup<IMM>(x1, c, sel[2]), lookup<IMM>(x0, c, sel[3]),
         lookup<IMM>(x1, c, sel[3]), bsel);
  mma_u8(a[0], a[1], a[2], a[3], lookup<IMM + 128u>(y0, c, sel[0]), lookup<IMM + 128u>(y1, c, sel[0]),
         lookup<IMM + 128u>(y0, c, sel[1]), lookup<IMM + 128u>(y1, c, sel[1]), bsel);
  mma_u8(b[0], b[1], b[2], b[3], lookup<IMM + 128u>(y0, c, sel[2]), lookup<IMM + 128u>(y1, c, sel[2]),
         lookup<IMM + 128u>(y0, c, sel[3]), lookup<IMM + 128u>(y1, c, sel[3]), bsel);
}

template <int W, int DEPTH, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 1)
lut_smem_kernel(const __grid_constant__ SbBatch batch, int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  using S = Shape<W, DEPTH, WARPS>;
  constexpr uint32_t SLOT = S::kSlot, kTableAddr = S::kTableAddr;
  constexpr int kThreads = S::kThreads;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3, hl = g >> 2, rot = g & 3;
  const uint32_t dyn = smem_u32(smem);
  if (dyn + kMiscBytes + S::kRingBytes > kTableAddr) {
    if (tid == 0 && status) atomicExch(status, (int)LCD_ERR_UNSUPPORTED);   // the window is not laid out as assumed
    return;
  }
  const uint32_t ring0 = dyn + kMiscBytes + (uint32_t)(warp * DEPTH) * SLOT;
  const uint32_t bar0 = dyn + 8u * (uint32_t)(warp * DEPTH);
  float* s_part = reinterpret_cast<float*>(smem + WARPS * DEPTH * 8);          // [WARPS]
  static_assert(WARPS * DEPTH * 8 + WARPS * 4 + 4 <= kMiscBytes, "barriers, maxima and the go flag");
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8u * i));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // the CTA's piece of the work sequence
  const uint2 st0 = batch.start[blockIdx.x], st1 = batch.start[blockIdx.x + 1];
  Piece geo{batch, (int)(st1.x >> 16), (int)(st1.x & 0xffffu), (int)st1.y};
  const int p0 = (int)(st0.x >> 16), s0 = (int)(st0.x & 0xffffu), rp0 = (int)st0.y;
  const bool has_work = !geo.at_end(p0, s0, rp0);

  // per-lane constants of the lookups
  uint32_t sel[4], c_first = 0, c_second = 0;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const uint32_t r = (uint32_t)((s + rot) & 3);
    sel[s] = 0xCC00u | (r << 4) | (uint32_t)(4 + s);
    c_first |= (4u * (uint32_t)(16 * hl + 4 * t) + 4u * r) << (8 * s);
    c_second |= (4u * (uint32_t)(16 * (1 - hl) + 4 * t) + 4u * r) << (8 * s);
  }
  const uint32_t bsel = g < 4 ? 1u << (8 * g) : 0u;     // B fragment: k-row 4t + i feeds column i

  // ---- fetch side of the ring: runs ahead of the consumer over the same walk -------------------------
  // A warp takes every WARPS-th row group of every segment (problem, slice) of the piece.  Inside a segment the next
  // row group is a fixed stride further in memory; the slice's geometry is worked out once per segment.
  uint64_t stream_policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
  int f_p = p0, f_s = s0, f_rp = rp0 + warp, f_rp_end = 0;
  bool f_live = has_work;
  uint32_t f_slot = 0, f_inflight = 0, f_bytes = 0;
  const uint8_t* f_src = nullptr;
  size_t f_stride = 0;
  auto f_enter = [&]() {      // settles on the first segment from (f_p, f_s) in which this warp has a row group
    while (f_live) {
      const int rp_end = geo.seg_end(f_p, f_s);
      if (f_rp < rp_end) {
        const SbProblem& P = batch.p[f_p];
        int kt0, width;
        slice_range(P, f_s, &kt0, &width);
        f_rp_end = rp_end;
        f_bytes = (uint32_t)width * kItemBytes;
        f_src = P.items + ((size_t)f_rp * P.n_kt + kt0) * kItemBytes;
        f_stride = (size_t)WARPS * P.n_kt * kItemBytes;
        return;
      }
      f_live = geo.next_segment(f_p, f_s);
      f_rp = warp;
    }
  };
  f_enter();
  auto fetch_one = [&]() {
    if (!f_live) return;
    if (lane == 0) {
      const uint32_t bar = bar0 + 8u * f_slot;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(f_bytes) : "memory");
      // weights are read once: evict-first keeps them from displacing what every CTA and every launch re-reads
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
          ::"r"(ring0 + f_slot * SLOT), "l"(f_src), "r"(f_bytes), "r"(bar), "l"(stream_policy) : "memory");
    }
    f_slot = f_slot + 1 == (uint32_t)DEPTH ? 0u : f_slot + 1;
    ++f_inflight;
    f_src += f_stride;
    f_rp += WARPS;
    if (f_rp >= f_rp_end) {
      f_live = geo.next_segment(f_p, f_s);
      f_rp = warp;
      f_enter();
    }
  };

  // Weights do not depend on the previous kernel of the stream: one stage per warp is queued before the dependency
  // wait, the others right behind the first requests for the activations (an SM's loads return in the order they
  // were queued, and the small ones must not wait behind the whole ring).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (has_work && batch.p[p0].act_bits == 16) {
    // ask the token and its smoothing factors into L2 (the weight stream evicts them between launches); a prefetch
    // cannot read stale data, L2 is the point of coherence
    const SbProblem& P = batch.p[p0];
    for (int k = tid * 64; k < P.K; k += kThreads * 64) {
      asm volatile("prefetch.global.L2 [%0];" ::"l"(P.x + k));
      if (P.inv_smooth) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(P.inv_smooth + k));
        if (k + 32 < P.K) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.inv_smooth + k + 32));
      }
    }
  }
  fetch_one();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  bool ring_primed = false;

  uint32_t c_slot = 0, c_phase = 0;
  bool aborted = false;
  int cur_p = -1;
  float amax = 0.0f;          // fused: the token's max |x * inv_s| of problem cur_p
  int seg_p = p0, seg_s = s0, seg_rp = rp0;
  bool seg_live = has_work;

#pragma unroll 1
  while (seg_live) {
    const SbProblem& P = batch.p[seg_p];
    int kt0, width;
    slice_range(P, seg_s, &kt0, &width);
    const int rp_end = geo.seg_end(seg_p, seg_s);
    const bool fused = P.act_bits == 16;

    // The columns of this thread's (first) table task, asked for together with the loads of the maximum below so
    // that the build does not pay a second trip to memory: task (block b, half-row hp, entry quarter i3), lane = bank.
    auto task_column = [&](int task) {
      const int b = task >> 3, hp = (task >> 2) & 1;
      const int G = 32 * (lane >> 4) + 8 * ((lane >> 2) & 3) + 4 * hp + (lane & 3);
      return (kt0 + b) * 256 + 4 * G;
    };
    float xv[4] = {0.0f, 0.0f, 0.0f, 0.0f}, fv[4] = {1.0f, 1.0f, 1.0f, 1.0f};
    uint32_t lv = 0x8888u;                       // non-fused: four stored levels
    auto load_columns = [&](int k) {
      if (fused) {
        if (P.x_vec && k < P.K) {           // K % 8 == 0: the four columns are inside together
          const uint2 raw = *reinterpret_cast<const uint2*>(P.x + k);
          const float2 v01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
          const float2 v23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
          xv[0] = v01.x; xv[1] = v01.y; xv[2] = v23.x; xv[3] = v23.y;
          if (P.inv_smooth) {
            const float4 f4 = __ldg(reinterpret_cast<const float4*>(P.inv_smooth + k));
            fv[0] = f4.x; fv[1] = f4.y; fv[2] = f4.z; fv[3] = f4.w;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            xv[j] = k + j < P.K ? __half2float(P.x[k + j]) : 0.0f;
            fv[j] = (k + j < P.K && P.inv_smooth) ? __ldg(P.inv_smooth + k + j) : 1.0f;
          }
        }
      } else {
        lv = __ldg(reinterpret_cast<const unsigned short*>(P.act_idx + (k >> 1)));
      }
    };
    if (warp < width * 8) load_columns(task_column(warp));

    // ---- Section 4.1 for this problem's token (each CTA for itself; x is a few KB in L2) ---------------
    if (seg_p != cur_p) {
      cur_p = seg_p;
      if (fused) {
        float m = 0.0f;
        if (P.x_vec) {
          for (int k = tid * 8; k < P.K; k += kThreads * 8) {
            const uint4 raw = *reinterpret_cast<const uint4*>(P.x + k);
            const __half2* h = reinterpret_cast<const __half2*>(&raw);
            float f[8];
            if (P.inv_smooth) {
              const float4 a = __ldg(reinterpret_cast<const float4*>(P.inv_smooth + k));
              const float4 b = __ldg(reinterpret_cast<const float4*>(P.inv_smooth + k + 4));
              f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) f[i] = 1.0f;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 v = __half22float2(h[i]);
              m = fmaxf(m, fmaxf(fabsf(__fmul_rn(v.x, f[2 * i])), fabsf(__fmul_rn(v.y, f[2 * i + 1]))));
            }
          }
        } else {
          for (int k = tid; k < P.K; k += kThreads)
            m = fmaxf(m, fabsf(__fmul_rn(__half2float(P.x[k]), P.inv_smooth ? __ldg(P.inv_smooth + k) : 1.0f)));
        }
        if (!ring_primed) {
          for (int i = 1; i < DEPTH; ++i) fetch_one();
          ring_primed = true;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        __syncthreads();                        // the previous problem's maxima have been read
        if (lane == 0) s_part[warp] = m;
        __syncthreads();
        amax = 0.0f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) amax = fmaxf(amax, s_part[w]);
        if (tid == 0) __stcg(batch.sq + seg_p, amax > 0.0f ? __fdiv_rn(amax, 7.0f) : 1.0f);   // for the rows' last step
      }
    }

    // ---- tables of the slice ------------------------------------------------------------------------------
    {
      const float r = amax > 0.0f ? __fdiv_rn(7.0f, amax) : 0.0f;
#pragma unroll 1
      for (int task = warp; task < width * 8; task += WARPS) {
        const int b = task >> 3, hp = (task >> 2) & 1, i3 = task & 3;
        if (task != warp) load_columns(task_column(task));
        uint32_t a[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (fused) {
            const float q = fminf(fmaxf(rintf(__fmul_rn(__fmul_rn(xv[j], fv[j]), r)), -8.0f), 7.0f);
            a[j] = (uint32_t)((int)q + 8);
          } else {
            a[j] = (lv >> (4 * j)) & 0xfu;
          }
        }
        // A[j][i]: column j falls into bucket i: byte i = its level, the other bytes 8
        uint32_t A[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) A[j][i] = (0x08080808u & ~(0xffu << (8 * i))) | (a[j] << (8 * i));
        uint32_t* dst = reinterpret_cast<uint32_t*>(smem + (kTableAddr - dyn) + (size_t)b * kBlockBytes +
                                                    (size_t)i3 * 64 * 256 + hp * 128 + lane * 4);
        uint32_t a3 = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) a3 = i3 == i ? A[3][i] : a3;
#pragma unroll
        for (int i2 = 0; i2 < 4; ++i2) {
          const uint32_t e2 = a3 + A[2][i2];
#pragma unroll
          for (int i1 = 0; i1 < 4; ++i1) {
            const uint32_t e1 = e2 + A[1][i1];
#pragma unroll
            for (int i0 = 0; i0 < 4; ++i0) dst[(i2 * 16 + i1 * 4 + i0) * 64] = e1 + A[0][i0];
          }
        }
      }
    }
    if (!ring_primed) {
      for (int i = 1; i < DEPTH; ++i) fetch_one();
      ring_primed = true;
    }
    __syncthreads();

    // ---- this warp's row groups of the segment: seg_rp + warp, + WARPS, ... ------------------------------
    const int bias = 32 * 64 * width;           // every table byte carries + 32, a row takes 64 lookups per block
    const int rp_first = seg_rp + warp;
    if (!aborted) {
      float* dst = P.sums + ((size_t)rp_first * 16 + g) * 4 + (t == 1 ? 32 : 0);
#pragma unroll 1
      for (int rp = rp_first; rp < rp_end; rp += WARPS) {
        if (!__all_sync(0xffffffffu, mbar_wait(bar0 + 8u * c_slot, c_phase))) { aborted = true; break; }
        const uint32_t item0 = ring0 + c_slot * SLOT + 16u * (uint32_t)lane;
        int acc[4] = {0, 0, 0, 0}, acc2[4] = {0, 0, 0, 0};    // two chains of dependent MMAs
#pragma unroll
        for (int b = 0; b < W; ++b) {
          if (b < width) {
            const uint32_t it = item0 + (uint32_t)b * kItemBytes;
            const uint4 r0 = lds128(it), r1 = lds128(it + 512u);        // this lane's 16 bytes of both tiles
            // k-block hl first, the other one second
            const uint32_t f0x = hl ? r0.z : r0.x, f0y = hl ? r0.w : r0.y, g0x = hl ? r0.x : r0.z, g0y = hl ? r0.y : r0.w;
            const uint32_t f1x = hl ? r1.z : r1.x, f1y = hl ? r1.w : r1.y, g1x = hl ? r1.x : r1.z, g1y = hl ? r1.y : r1.w;
            if (b == 0) {
              half_item<kTableAddr>(f0x, f0y, f1x, f1y, c_first, sel, bsel, acc, acc2);
              half_item<kTableAddr>(g0x, g0y, g1x, g1y, c_second, sel, bsel, acc, acc2);
            } else if (b == 1) {
              half_item<kTableAddr + kBlockBytes>(f0x, f0y, f1x, f1y, c_first, sel, bsel, acc, acc2);
              half_item<kTableAddr + kBlockBytes>(g0x, g0y, g1x, g1y, c_second, sel, bsel, acc, acc2);
            } else {
              half_item<kTableAddr + 2u * kBlockBytes>(f0x, f0y, f1x, f1y, c_first, sel, bsel, acc, acc2);
              half_item<kTableAddr + 2u * kBlockBytes>(g0x, g0y, g1x, g1y, c_second, sel, bsel, acc, acc2);
            }
          }
        }
        --f_inflight;
        if (++c_slot == (uint32_t)DEPTH) { c_slot = 0; c_phase ^= 1u; }
        // lanes t = 0, 1 hold buckets 2t, 2t + 1 of rows g and g + 8
        const float f0 = (float)(acc[0] + acc2[0] - bias), f1 = (float)(acc[1] + acc2[1] - bias);
        const float f2 = (float)(acc[2] + acc2[2] - bias), f3 = (float)(acc[3] + acc2[3] - bias);
        // lane t = 0 collects the four buckets of row g, lane t = 1 those of row g + 8
        const float x0 = __shfl_xor_sync(0xffffffffu, t == 0 ? f2 : f0, 1);
        const float x1 = __shfl_xor_sync(0xffffffffu, t == 0 ? f3 : f1, 1);
        fetch_one();       // the sums are formed, so every read of the slot has completed: it may be refilled
        if (t == 0) red_add_v4(dst, f0, f1, x0, x1);
        if (t == 1) red_add_v4(dst, x0, x1, f2, f3);
        dst += (size_t)WARPS * 64;
      }
      if (aborted && lane == 0 && status) atomicExch(status, (int)LCD_ERR_TIMEOUT);
    }
    seg_live = geo.next_segment(seg_p, seg_s);
    seg_rp = 0;
    if (seg_live) __syncthreads();     // every warp is done with the tables before they are rebuilt
  }
  if (aborted) {      // copies already issued must land before the CTA may exit
    while (f_inflight > 0) {
      (void)mbar_wait(bar0 + 8u * c_slot, c_phase);
      --f_inflight;
      if (++c_slot == (uint32_t)DEPTH) { c_slot = 0; c_phase ^= 1u; }
    }
  }

  // ---- every CTA's sums must be in the scratch before a row can be finished ---------------------------------
  // The rows of all problems are dealt to all threads of the grid; a thread's first row and its centroids do not
  // depend on the sums and are fetched before the wait.
  const int total_rows = batch.row0[batch.count];
  auto locate = [&](int r, int* n) {
    int p = 0;
#pragma unroll
    for (int i = 1; i < LCD_MAX_BATCH; ++i) p = (i < batch.count && r >= batch.row0[i]) ? i : p;
    *n = r - batch.row0[p];
    return p;
  };
  int r = (int)blockIdx.x * kThreads + tid;
  int n_cur = 0, p_cur = 0;
  uint2 c_cur = make_uint2(0u, 0u);
  if (r < total_rows) {
    p_cur = locate(r, &n_cur);
    c_cur = __ldg(reinterpret_cast<const uint2*>(batch.p[p_cur].codebook + (size_t)n_cur * 4));
  }
  int& s_go = *reinterpret_cast<int*>(smem + WARPS * DEPTH * 8 + WARPS * 4);   // in the misc area: no static shared memory
  __threadfence();                       // this thread's reductions are performed
  __syncthreads();
  if (tid == 0) {
    int go = 1;
    atomicAdd(batch.gate, 1);
    const unsigned long long t0 = globaltimer();
    for (uint32_t it = 0;; ++it) {
      int seen;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(batch.gate) : "memory");
      if (seen >= (int)gridDim.x) break;
      if ((it & 63u) == 63u && globaltimer() - t0 > kTimeoutNs) { go = 0; break; }
      __nanosleep(32);
    }
    s_go = go;
  }
  __syncthreads();
  if (!s_go) {
    if (tid == 0 && status) atomicExch(status, (int)LCD_ERR_TIMEOUT);
    return;
  }
  for (; r < total_rows; r += (int)gridDim.x * kThreads) {
    const SbProblem& P = batch.p[p_cur];
    float4* src = reinterpret_cast<float4*>(P.sums) + n_cur;
    const float4 Sw = __ldcg(src);
    const float sq = P.act_bits == 16 ? __ldcg(batch.sq + p_cur) : __ldg(P.act_scale);
    __stcg(src, make_float4(0.0f, 0.0f, 0.0f, 0.0f));          // handed on zero-filled
    const float2 c01 = __half22float2(*reinterpret_cast<const __half2*>(&c_cur.x));
    const float2 c23 = __half22float2(*reinterpret_cast<const __half2*>(&c_cur.y));
    const float v = (c01.x * Sw.x + c01.y * Sw.y) + (c23.x * Sw.z + c23.y * Sw.w);
    if (n_cur < P.N) P.y[n_cur] = v * sq;
    const int r_next = r + (int)gridDim.x * kThreads;
    if (r_next < total_rows) {
      p_cur = locate(r_next, &n_cur);
      c_cur = __ldg(reinterpret_cast<const uint2*>(batch.p[p_cur].codebook + (size_t)n_cur * 4));
    }
  }
  // the CTA that leaves last clears the counters and the scales
  __syncthreads();
  if (tid == 0 && atomicAdd(batch.gate + 1, 1) == (int)gridDim.x - 1) {
    for (int i = 0; i < LCD_MAX_BATCH; ++i) __stcg(batch.sq + i, 0.0f);
    atomicExch(batch.gate, 0);
    atomicExch(batch.gate + 1, 0);
  }
}

int sm_count_now() { return current_sm_count(); }

constexpr int kSliceBlocks = 2;    // W: table blocks per slice (2 x 64 KB)
constexpr int kDepth = 2;          // ring slots per warp: 64 KB in flight per SM (three measured no faster, the first
                                   // loads of a launch wait behind the ring's first fill)
constexpr int kWarps = 16;
using LaunchShape = Shape<kSliceBlocks, kDepth, kWarps>;

int slices_of(int64_t n_kt) { return (int)((n_kt + kSliceBlocks - 1) / kSliceBlocks); }

// Scratch of a launch: 256 bytes of counters and scales, then every problem's bucket sums.
constexpr size_t kGateBytes = 256;
size_t sums_bytes(const Problem& p) { return (size_t)round_up_u64((uint64_t)p.N_pad * 4 * sizeof(float), 256); }

}  // namespace

bool lut_smem_supported(const Problem* probs, int count) {
  if (count < 1 || count > LCD_MAX_BATCH) return false;
  for (int i = 0; i < count; ++i) {
    const Problem& p = probs[i];
    if (p.M != 1 || p.bits != 2 || (p.act_bits != 4 && p.act_bits != 16)) return false;
    if (p.N_pad >= (1 << 27) || p.K_pad / kTileK >= (1 << 15)) return false;
    if (p.K_pad > (1 << 20)) return false;      // bucket sums stay below 2^24: exact in fp32
  }
  return true;
}

size_t lut_smem_workspace_bytes(const Problem* probs, int count) {
  size_t off = kGateBytes;
  for (int i = 0; i < count; ++i) off += sums_bytes(probs[i]);
  return off;
}

lcd_status launch_lut_smem(const Problem* probs, int count, void* workspace, size_t workspace_bytes, int32_t* status_word,
                           void* stream) {
  if (!lut_smem_supported(probs, count)) return LCD_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < lut_smem_workspace_bytes(probs, count)) return LCD_ERR_BUFFER_TOO_SMALL;
  SbBatch batch;
  batch.count = count;
  batch.gate = reinterpret_cast<int*>(workspace);
  batch.sq = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + 64);
  batch.row0[0] = 0;
  size_t off = kGateBytes;
  for (int i = 0; i < count; ++i) {
    const Problem& p = probs[i];
    SbProblem& g = batch.p[i];
    g.items = p.tiles;
    g.codebook = p.codebook;
    g.act_idx = p.act_idx;
    g.act_scale = p.act_scale;
    g.x = static_cast<const __half*>(p.x_fp16);
    g.inv_smooth = p.inv_smooth;
    g.y = p.y;
    g.sums = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + off);
    off += sums_bytes(p);
    batch.row0[i + 1] = batch.row0[i] + (int)p.N_pad;
    g.K = (int)p.K;
    g.N = (int)p.N;
    g.N_pad = (int)p.N_pad;
    g.n_rp = (int)(p.N_pad / kPairRows);
    g.n_kt = (int)(p.K_pad / kTileK);
    g.n_slices = slices_of(g.n_kt);
    g.act_bits = p.act_bits;
    g.x_vec = (p.K % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.x_fp16) & 15) == 0) &&
              (!p.inv_smooth || (reinterpret_cast<uintptr_t>(p.inv_smooth) & 15) == 0);
  }
  for (int i = count; i < LCD_MAX_BATCH; ++i) { batch.p[i] = batch.p[0]; batch.row0[i + 1] = batch.row0[count]; }

  // Cut the sequence (problem, slice, row group) into one contiguous piece per CTA.  A piece costs its items plus,
  // for every slice it touches, the table build (in items, measured); the smallest cost limit that fits into the
  // CTAs is found by bisection over a greedy sweep.
  const int n_cta = sm_count_now() < kMaxCta ? sm_count_now() : kMaxCta;
  // Costs in units of 9 ns (measured): a row group takes 27 ns plus 18 ns per item (3 + 2 * width), a segment's
  // tables 1.2 us, the token's maximum of another problem 0.9 us plus 0.1 us per 1024 columns, the barriers around a
  // rebuild and the warps' uneven ends 1.5 us.
  auto group_cost = [](int width) { return 3 + 2 * width; };
  auto build_cost = [](int width, bool first, int new_problem_K) {
    return 30 + 50 * width + (first ? 0 : 165) + (new_problem_K > 0 ? 100 + new_problem_K / 90 : 0);
  };
  auto sweep = [&](long long limit, uint2* start) -> int {
    int cta = 0, last_p = -1;   // last_p: problem of the current CTA's latest segment
    long long used = 0;
    bool open = false;          // the current CTA already has work
    for (int p = 0; p < count; ++p) {
      const SbProblem& g = batch.p[p];
      for (int s = 0; s < g.n_slices; ++s) {
        const int width = (int)((long long)(s + 1) * g.n_kt / g.n_slices - (long long)s * g.n_kt / g.n_slices);
        int rp = 0;
        while (rp < g.n_rp) {
          const int fixed = build_cost(width, !open, (!open || last_p != p) ? g.K : 0);
          long long room = (limit - used - fixed) / group_cost(width);
          if (room < 1 && open) {      // no room for even one row group of this slice: next CTA
            ++cta;
            used = 0;
            open = false;
            continue;
          }
          if (room < 1) room = 1;
          if (!open) {
            if (start && cta <= kMaxCta) start[cta] = make_uint2((unsigned)p << 16 | (unsigned)s, (unsigned)rp);
            open = true;
          }
          const int take = (int)(room < g.n_rp - rp ? room : g.n_rp - rp);
          used += fixed + (long long)take * group_cost(width);
          last_p = p;
          rp += take;
          if (rp < g.n_rp) {           // the slice continues in the next CTA
            ++cta;
            used = 0;
            open = false;
          }
        }
      }
    }
    return cta + (open ? 1 : 0);
  };
  long long total = 0, lo = 1, hi;
  for (int p = 0; p < count; ++p)
    total += (long long)batch.p[p].n_rp * batch.p[p].n_slices * group_cost(kSliceBlocks) +
             (long long)batch.p[p].n_slices * build_cost(kSliceBlocks, false, batch.p[p].K);
  hi = total + build_cost(kSliceBlocks, false, 1 << 20) + group_cost(kSliceBlocks);
  while (lo < hi) {
    const long long mid = (lo + hi) / 2;
    if (sweep(mid, nullptr) <= n_cta) hi = mid; else lo = mid + 1;
  }
  const int used = sweep(lo, batch.start);
  for (int c = used; c <= kMaxCta; ++c) batch.start[c] = make_uint2((unsigned)count << 16, 0u);
  batch.n_cta = used;

  auto kern = lut_smem_kernel<kSliceBlocks, kDepth, kWarps>;
  static PerDeviceFlag attr_set;
  int dev;
  if (attr_set.first(&dev)) {
    const cudaError_t ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LaunchShape::kSmemBytes);
    if (ea != cudaSuccess) { set_cuda_error((int)ea); return LCD_ERR_CUDA; }
    attr_set.done(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)used);
  cfg.blockDim = dim3(LaunchShape::kThreads);
  cfg.dynamicSmemBytes = LaunchShape::kSmemBytes;
  cfg.stream = static_cast<cudaStream_t>(stream);
  // cooperative: all CTAs wait for one another before the rows are finished, so all of them must be resident
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeCooperative;
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, batch, status_word);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
