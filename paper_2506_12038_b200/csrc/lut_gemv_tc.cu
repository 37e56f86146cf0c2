// LUT-GEMV for M <= 16 tokens on the tcgen05 tensor cores (LCD_ALGO_TC_LUT).
//
// Same arithmetic as the register-LUT kernel (Section 4.2 of the LCD paper: per row two byte tables, 16-bit fixed
// point, looked up four weights at a time with PRMT; exact int32 sums of table byte x activation level;
// y = s_q * 2^e_n * (256 * sumH + sumL)), but the looked-up bytes are written straight from registers into
// tensor memory (tcgen05.st) as the A operand of tcgen05.mma kind::i8, whose B operand is the 16-token tile of
// levels in shared memory.  Nothing of the decoded weights passes through shared memory and no warp-level MMA,
// fragment load or per-row combine is issued by the decoding warps.
//
// Work: the 128-row x 256-column units (8 items) of all problems of the launch form one sequence that is cut evenly
// over the CTAs (one per SM); a row tile whose columns are shared by several CTAs is summed with integer atomics in
// zero-filled global scratch, the last arrival (ticket) writes y and leaves zeros.  Integer accumulation is order
// free, so several threads issue MMAs into one accumulator that the epilogue zero-fills after every use.
//
// Warps: 0-5 MMA issuers (one per stage slot), 6-9 epilogue (tensor-memory quadrant each), 10-25 decoders = 4 groups
// (unit number mod 4) x 4 quadrant warps; a decoder thread owns one row, its warp streams its 32 rows' items through
// a private shared-memory ring filled by cp.async.bulk, and the 128 threads of a group also stage the stage's
// 16 x 128 token levels (4-bit -> int8 in lookup order -> swizzled shared-memory tile, one 16-byte chunk each).  Every wait is bounded; on expiry the status word is set and all roles
// leave their loops, drain what they issued and release tensor memory.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "device_util.h"

namespace lcd {

namespace {

constexpr int kTcTokens = 16;                 // MMA N: tokens per tile (rows past M are zero)
constexpr int kTcRows = 128;                  // MMA M: weight rows per tile
constexpr int kTcSlots = 6;                   // pipeline stages (128 columns each): A in tensor memory, B in smem
constexpr int kTcIssuers = kTcSlots, kTcEpi = 4, kTcDecoders = 16;
constexpr int kTcFirstIssuer = 0, kTcFirstEpi = kTcFirstIssuer + kTcIssuers;
constexpr int kTcFirstDecoder = kTcFirstEpi + kTcEpi;
constexpr int kTcThreads = 32 * (kTcFirstDecoder + kTcDecoders);     // 832
constexpr int kTcRing = 3;                    // ring slots per decoder warp (one 256-column unit of its 32 rows each)
constexpr int kTcBBytes = kTcTokens * 128;    // 2 KB: 16 tokens x 128 int8
constexpr uint32_t kTcACols = 64;             // tensor-memory columns of one A stage: 32 high plane + 32 low plane
constexpr uint32_t kTcAccCol0 = kTcSlots * kTcACols;   // accumulators: 2 buffers x (16 high + 16 low) columns
constexpr unsigned long long kTcWaitNs = 500000000ull;   // no legitimate wait is longer than milliseconds

struct TcProblem {
  const uint8_t* items;
  const uint16_t* codebook;
  const uint8_t* act_idx;
  const float* act_scale;
  float* y;
  int* acc;        // scratch [n_rt][2 planes][16 tokens][128 rows] int32, zero on entry and on exit
  int* ticket;     // scratch [n_rt][4 quadrants] int32, zero on entry and on exit
  long long ldy;
  int N, M, n_rp, n_kt, n_rt;
  int act_bits;    // 4: act_idx is [M][K_pad/2] packed levels + 8; 8: [M][K_pad] signed bytes
  unsigned unit0;  // number of units of the problems before this one
};
struct TcBatch {
  int count;
  unsigned total_units;
  TcProblem p[LCD_MAX_BATCH];
};

__device__ __forceinline__ uint32_t tc_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ unsigned long long tc_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool tc_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  SLEEP: the thread sleeps between polls (roles that wait long and are not on the critical path: the
// epilogue), so that it leaves the issue slots to the others; otherwise it polls back to back, because the wake-up
// delay of a sleeping thread would be added to every hand-over of a pipeline stage.
template <bool SLEEP = false>
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (tc_try(bar, parity)) return true;
  const unsigned long long t0 = tc_timer();
#pragma unroll 1
  for (uint32_t it = 1;; ++it) {
    if (SLEEP) __nanosleep(200);
    if (tc_try(bar, parity)) return true;
    if ((it & (SLEEP ? 63u : 1023u)) == 0) {
      if (*abort_flag) return false;
      if (tc_timer() - t0 > kTcWaitNs) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void tc_drain(uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = tc_timer();
  for (uint32_t it = 1; !tc_try(bar, parity); ++it)
    if ((it & 255u) == 0 && tc_timer() - t0 > kTcWaitNs) return;
}
__device__ __forceinline__ void tc_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// kind::i8, A from tensor memory, B from shared memory (K-major, 128-byte swizzle), always accumulating.
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, 1, 0;\ntcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc) : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
}
// kind::i8 instruction descriptor: int32 accumulate, B signed, A signed (high plane) or unsigned (low plane)
__host__ __device__ constexpr uint32_t tc_idesc(bool a_signed) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(kTcTokens >> 3) << 17) |
         ((uint32_t)(kTcRows >> 4) << 24);
}
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
  uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Position in the sequence of units (128 rows x 256 columns) of the launch: problem, row tile, column unit.
struct Walk {
  uint32_t u;      // global unit number
  int p, rt, kt;
  int n_kt, n_rt;  // of problem p (kept here: indexing the kernel parameters at every step is slow)
};
__device__ __forceinline__ void walk_set(Walk& w, uint32_t u, const TcBatch& B) {
  w.u = u;
  w.p = 0;
  for (int i = 1; i < B.count; ++i)
    if (u >= B.p[i].unit0) w.p = i;
  w.n_kt = B.p[w.p].n_kt;
  w.n_rt = B.p[w.p].n_rt;
  const uint32_t local = u - B.p[w.p].unit0;
  w.rt = (int)(local / (uint32_t)w.n_kt);
  w.kt = (int)(local - (uint32_t)w.rt * (uint32_t)w.n_kt);
}
__device__ __forceinline__ void walk_step(Walk& w, const TcBatch& B) {
  ++w.u;
  if (++w.kt == w.n_kt) {
    w.kt = 0;
    if (++w.rt == w.n_rt) {
      w.rt = 0;
      if (w.p + 1 < B.count) {
        ++w.p;
        w.n_kt = B.p[w.p].n_kt;
        w.n_rt = B.p[w.p].n_rt;
      }
    }
  }
}

// CTA c of G owns the units [c * T / G, (c + 1) * T / G); the CTA that owns unit u.
__device__ __forceinline__ uint32_t unit_begin(uint32_t c, uint32_t G, uint32_t T) {
  return (uint32_t)(((unsigned long long)c * T) / G);
}
__device__ __forceinline__ uint32_t unit_owner(uint32_t u, uint32_t G, uint32_t T) {
  // largest c with floor(c * T / G) <= u
  uint32_t c = (uint32_t)((((unsigned long long)u + 1) * G - 1) / T);
  while (c + 1 < G && unit_begin(c + 1, G, T) <= u) ++c;
  while (c > 0 && unit_begin(c, G, T) > u) --c;
  return c;
}

template <int BITS>
__global__ void __launch_bounds__(kTcThreads, 1) lut_gemv_tc_kernel(const TcBatch B, int* status) {
  extern __shared__ uint8_t tc_smem_raw[];
  constexpr int ITEM = 512 * BITS, HALF = 256 * BITS;
  constexpr int kSlotBytes = 2 * ITEM;                              // the two 16-row groups of a warp's 32 rows
  constexpr int kRingBytes = kTcDecoders * kTcRing * kSlotBytes;
  constexpr uint32_t kTmemCols = 512;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t raw_addr = (uint32_t)__cvta_generic_to_shared(tc_smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* gen_base = tc_smem_raw + (base - raw_addr);
  // [ token tiles: kTcSlots x 2 KB | rings | barriers | misc ]
  const uint32_t ring_base = base + kTcSlots * kTcBBytes;
  const uint32_t bar_base = ring_base + kRingBytes;
  auto full = [&](int s) { return bar_base + 8u * s; };
  // A stage slot is filled by different decoder groups in turn, so a group skips uses of a slot.  One release
  // barrier per slot would let a group that waits for use n - 1 be two phases ahead of it, where a parity wait
  // passes at once; with one barrier per slot and use parity every waiter is at most one phase ahead.
  auto empty = [&](int s, uint32_t use) { return bar_base + 8u * (kTcSlots + 2 * s + (int)(use & 1u)); };
  auto tmem_full = [&](int b) { return bar_base + 8u * (3 * kTcSlots + b); };
  auto tmem_empty = [&](int b) { return bar_base + 8u * (3 * kTcSlots + 2 + b); };
  const uint32_t drain_bar = bar_base + 8u * (3 * kTcSlots + 4);
  auto ring_bar = [&](int dw, int s) { return bar_base + 8u * (3 * kTcSlots + 5 + dw * kTcRing + s); };
  constexpr int kNumBars = 3 * kTcSlots + 5 + kTcDecoders * kTcRing;
  uint8_t* gen_misc = gen_base + kTcSlots * kTcBBytes + kRingBytes + 8 * kNumBars;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(gen_misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_misc + 4);
  // wait until stage number `it` may overwrite its slot: use n = it / kTcSlots needs use n - 1 consumed
  auto wait_slot_free = [&](uint32_t it) {
    const uint32_t use = it / kTcSlots;
    if (use == 0) return true;
    return tc_wait(empty((int)(it % kTcSlots), use - 1), ((use - 1) >> 1) & 1u, abort_flag);
  };

  // token tiles start as zeros: rows of tokens a problem does not have are never written
  for (int i = threadIdx.x; i < kTcSlots * kTcBBytes / 16; i += kTcThreads)
    reinterpret_cast<uint4*>(gen_base)[i] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    auto init = [](uint32_t bar, uint32_t count) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    };
    for (int s = 0; s < kTcSlots; ++s) {
      init(full(s), 4 * 32);             // one decoder group (4 warps)
      init(empty(s, 0), 1);              // the issuer of the stage
      init(empty(s, 1), 1);
    }
    for (int b = 0; b < 2; ++b) {
      init(tmem_full(b), kTcIssuers);
      init(tmem_empty(b), kTcEpi * 32);
    }
    init(drain_bar, kTcIssuers);
    for (int i = 0; i < kTcDecoders * kTcRing; ++i) init(ring_bar(0, i), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kTcFirstIssuer) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const uint32_t G = gridDim.x, T = B.total_units;
  const uint32_t u0 = unit_begin(blockIdx.x, G, T), u1 = unit_begin(blockIdx.x + 1, G, T);
  const uint32_t n_units = u1 - u0;

  if (warp < kTcFirstEpi) {
    // ------------------------------------------------------------------ MMA issuers
    // One thread per stage slot: a slot's fill barrier is then always waited on by the same thread, in order.
    if (lane == 0) {
      const uint32_t me = (uint32_t)(warp - kTcFirstIssuer);
      const uint32_t idesc_hi = tc_idesc(true), idesc_lo = tc_idesc(false);
      Walk w;
      if (n_units) walk_set(w, u0, B);
      bool ok = true;
      uint32_t sg = 0;
      bool seg_open = false;
      for (uint32_t ic = 0; ic < n_units && ok; ++ic) {
        const uint32_t buf = sg & 1u;
        if (!seg_open) {
          if (!tc_wait(tmem_empty(buf), (sg >> 1) & 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          seg_open = true;
        }
        const uint32_t d_hi = tmem_base + kTcAccCol0 + buf * 32u;
        if (ic % 3u == (me >> 1)) {                 // stage 2 * ic + h is this thread's when it is me modulo 6
          const uint32_t it = 2u * ic + (me & 1u);
          const int slot = (int)me;
          if (!tc_wait(full(slot), (it / kTcSlots) & 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t bd = tc_smem_desc(base + slot * kTcBBytes);
          const uint32_t a = tmem_base + slot * kTcACols;
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma(d_hi, a + 8 * k, bd + 2 * k, idesc_hi);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma(d_hi + 16, a + 32 + 8 * k, bd + 2 * k, idesc_lo);
          tc_commit(empty(slot, it / kTcSlots));
        }
        const bool last = (ic + 1 == n_units) || (w.kt + 1 == w.n_kt);
        if (last) {
          tc_commit(tmem_full(buf));
          seg_open = false;
          ++sg;
        }
        walk_step(w, B);
      }
      tc_commit(drain_bar);
      tc_drain(drain_bar, 0);
    }
    __syncwarp();
  } else if (warp < kTcFirstDecoder) {
    // ------------------------------------------------------------------ epilogue (one tensor-memory quadrant each)
    const int quad = warp & 3;
    const uint32_t lane_field = (uint32_t)(32 * quad) << 16;
    // zero both accumulator buffers, then hand them to the issuers
    {
      const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
      for (int c = 0; c < 8; ++c) tc_st8(tmem_base + lane_field + kTcAccCol0 + 8 * c, z);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      tc_arrive(tmem_empty(0));
      tc_arrive(tmem_empty(1));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    Walk w;
    if (n_units) walk_set(w, u0, B);
    bool ok = true;
    uint32_t sg = 0;
    int seg_kt0 = n_units ? w.kt : 0;
    for (uint32_t ic = 0; ic < n_units && ok; ++ic) {
      const bool last = (ic + 1 == n_units) || (w.kt + 1 == w.n_kt);
      if (last) {
        const TcProblem& P = B.p[w.p];
        const uint32_t buf = sg & 1u;
        const int row = 32 * quad + lane;
        const int n = w.rt * kTcRows + row;
        const int n_cb = n < P.n_rp * 16 ? n : P.n_rp * 16 - 1;
        float mx = 0.0f;
#pragma unroll
        for (int i = 0; i < (1 << BITS); ++i)
          mx = fmaxf(mx, fabsf(__half2float(__ushort_as_half(__ldg(P.codebook + (size_t)n_cb * (1 << BITS) + i)))));
        int ex = (int)((__float_as_uint(mx) >> 23) & 0xffu) - 126;
        ex = ex < -30 ? -30 : ex;
        const float row_scale = __uint_as_float((uint32_t)(ex - 15 + 127) << 23);   // 2^(e-15) of the row's tables
        const float my_scale = (lane < 16 && lane < P.M) ? __ldg(P.act_scale + lane) : 0.0f;
        ok = __all_sync(0xffffffffu, tc_wait<true>(tmem_full(buf), (sg >> 1) & 1u, abort_flag));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t hi[16], lo[16];
        const uint32_t t_hi = tmem_base + lane_field + kTcAccCol0 + buf * 32u;
        tc_ld16(t_hi, hi);
        tc_ld16(t_hi + 16, lo);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        // zero the buffer and give it back before the (slow) global part
        {
          const uint32_t z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
          for (int c = 0; c < 4; ++c) tc_st8(t_hi + 8 * c, z);
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          tc_arrive(tmem_empty(buf));
        }
        const bool whole = seg_kt0 == 0 && w.kt + 1 == P.n_kt;
        if (whole) {
#pragma unroll
          for (int j = 0; j < kTcTokens; ++j) {
            const float s = __shfl_sync(0xffffffffu, my_scale, j) * row_scale;
            if (j < P.M && n < P.N) P.y[(size_t)j * P.ldy + n] = ((float)(int)hi[j] * 256.0f + (float)(int)lo[j]) * s;
          }
        } else {
          int* acc = P.acc + (size_t)w.rt * (2 * kTcTokens * kTcRows) + row;
#pragma unroll
          for (int j = 0; j < kTcTokens; ++j)
            if (j < P.M) {
              atomicAdd(acc + j * kTcRows, (int)hi[j]);
              atomicAdd(acc + (kTcTokens + j) * kTcRows, (int)lo[j]);
            }
          __threadfence();
          __syncwarp();
          int is_last = 0;
          if (lane == 0) {
            const uint32_t ua = P.unit0 + (uint32_t)w.rt * (uint32_t)P.n_kt;
            const int expected = (int)(unit_owner(ua + (uint32_t)P.n_kt - 1, G, T) - unit_owner(ua, G, T)) + 1;
            const int t = atomicAdd(P.ticket + w.rt * 4 + quad, 1);
            is_last = (t == expected - 1);
            if (is_last) P.ticket[w.rt * 4 + quad] = 0;
          }
          is_last = __shfl_sync(0xffffffffu, is_last, 0);
          if (is_last) {
            __threadfence();
#pragma unroll
            for (int j = 0; j < kTcTokens; ++j) {
              const float s = __shfl_sync(0xffffffffu, my_scale, j) * row_scale;
              if (j < P.M) {
                const int vh = atomicExch(acc + j * kTcRows, 0);
                const int vl = atomicExch(acc + (kTcTokens + j) * kTcRows, 0);
                if (n < P.N) P.y[(size_t)j * P.ldy + n] = ((float)vh * 256.0f + (float)vl) * s;
              }
            }
          }
        }
        ++sg;
      }
      walk_step(w, B);
      if (last) seg_kt0 = w.kt;
    }
  } else {
    // ------------------------------------------------------------------ decoders
    // Group j takes the units j, j + 4, ... of the CTA (both 128-column stages of each); a thread owns one row:
    // tensor-memory lane 32 * quad + lane = row of the tile.  The warp's 32 rows are two 16-row items per unit,
    // streamed through the warp's ring by its lane 0.
    const int dw = warp - kTcFirstDecoder, grp = dw >> 2, quad = warp & 3;
    const int u = (lane >> 3) & 1, g = lane & 7;
    const uint32_t lane_field = (uint32_t)(32 * quad) << 16;
    const uint32_t my_ring = ring_base + (uint32_t)dw * kTcRing * kSlotBytes;
    const uint32_t n_own = n_units > (uint32_t)grp ? (n_units - (uint32_t)grp + 3u) / 4u : 0u;
    Walk wf, wc;
    if (n_own) { walk_set(wf, u0 + (uint32_t)grp, B); wc = wf; }
    auto fetch = [&](uint32_t oi) {          // lane 0: start the copies of own unit oi (wf is at that unit)
      const TcProblem& P = B.p[wf.p];
      const uint32_t slot = oi % kTcRing;
      const uint32_t bar = ring_bar(dw, (int)slot);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)kSlotBytes) : "memory");
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        int rp = wf.rt * (kTcRows / 16) + 2 * quad + i;
        rp = rp < P.n_rp ? rp : P.n_rp - 1;        // rows past the matrix repeat the last group; never stored
        const uint8_t* src = P.items + ((size_t)rp * P.n_kt + wf.kt) * ITEM;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(my_ring + slot * kSlotBytes + i * ITEM), "l"(src), "r"((uint32_t)ITEM), "r"(bar) : "memory");
      }
    };
    auto advance4 = [&](Walk& w) {
#pragma unroll 1
      for (int i = 0; i < 4; ++i) walk_step(w, B);
    };
    uint32_t fetched = 0;
    if (lane == 0)
      for (; fetched < n_own && fetched < (uint32_t)kTcRing; ++fetched) { fetch(fetched); advance4(wf); }

    // Each decoder thread also stages one 16-column piece of one token's levels per stage (128 threads = 16 tokens
    // x 8 pieces): 8 bytes of 4-bit levels become one 16-byte chunk of signed bytes in the lookup order.
    const int tk_token = (32 * quad + lane) >> 3, tk_piece = lane & 7;
    const uint8_t* act_ptr = nullptr;       // this thread's token row (+ piece), null when the problem has no such token
    bool act8 = false;                      // 8-bit levels: 16 bytes per piece, only their order changes
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint32_t TH[2] = {0, 0}, TL[2] = {0, 0};
    int tab_p = -1, tab_rt = -1;
    bool ok = true;
    uint32_t consumed = 0;
    for (uint32_t oi = 0; oi < n_own && ok; ++oi) {
      const TcProblem& P = B.p[wc.p];
      if (wc.p != tab_p || wc.rt != tab_rt) {
        // byte tables of this thread's row: 16-bit fixed point, high (signed) and low (unsigned) bytes
        tab_p = wc.p; tab_rt = wc.rt;
        act8 = P.act_bits == 8;
        act_ptr = tk_token < P.M ? P.act_idx + ((size_t)tk_token * ((size_t)P.n_kt * 128) + tk_piece * 8) * (act8 ? 2 : 1)
                                 : nullptr;
        int n = wc.rt * kTcRows + 32 * quad + lane;
        n = n < P.n_rp * 16 ? n : P.n_rp * 16 - 1;
        const uint16_t* cb = P.codebook + (size_t)n * (1 << BITS);
        float mx = 0.0f;
#pragma unroll
        for (int i = 0; i < (1 << BITS); ++i) mx = fmaxf(mx, fabsf(__half2float(__ushort_as_half(__ldg(cb + i)))));
        int ex = (int)((__float_as_uint(mx) >> 23) & 0xffu) - 126;
        ex = ex < -30 ? -30 : ex;
        const float up = __uint_as_float((uint32_t)(15 - ex + 127) << 23);
        TH[0] = TH[1] = TL[0] = TL[1] = 0u;
#pragma unroll
        for (int i = 0; i < (1 << BITS); ++i) {
          const int f = __float2int_rn(__half2float(__ushort_as_half(__ldg(cb + i))) * up);
          TH[i >> 2] |= ((uint32_t)(f >> 8) & 0xffu) << (8 * (i & 3));
          TL[i >> 2] |= ((uint32_t)f & 0xffu) << (8 * (i & 3));
        }
        if (BITS == 2) { TH[1] = TH[0]; TL[1] = TL[0]; }
      }
      uint4 lv[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      if (act_ptr) {
        if (act8) {
          lv[0] = __ldg(reinterpret_cast<const uint4*>(act_ptr + (size_t)wc.kt * 256));
          lv[1] = __ldg(reinterpret_cast<const uint4*>(act_ptr + (size_t)wc.kt * 256 + 128));
        } else {
          const uint2 a = __ldg(reinterpret_cast<const uint2*>(act_ptr + (size_t)wc.kt * 128));
          const uint2 b = __ldg(reinterpret_cast<const uint2*>(act_ptr + (size_t)wc.kt * 128 + 64));
          lv[0].x = a.x; lv[0].y = a.y; lv[1].x = b.x; lv[1].y = b.y;
        }
      }
      const uint32_t rslot = oi % kTcRing;
      // tcgen05.st below is warp-collective: the whole warp leaves a wait together
      ok = __all_sync(0xffffffffu, tc_wait(ring_bar(dw, (int)rslot), (oi / kTcRing) & 1u, abort_flag));
      if (!ok) break;
      consumed = oi + 1;
      const uint32_t src = my_ring + rslot * kSlotBytes + (uint32_t)((lane >> 4) * ITEM + u * HALF);
      uint32_t raw[4][BITS == 2 ? 4 : 6];            // [quarter t][k-block h x words]
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        if (BITS == 2) {
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(raw[t][0]), "=r"(raw[t][1]), "=r"(raw[t][2]), "=r"(raw[t][3])
                       : "r"(src + 16u * (uint32_t)(4 * g + t)));
        } else {
#pragma unroll
          for (int b = 0; b < 3; ++b)
            asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];"
                         : "=r"(raw[t][b]), "=r"(raw[t][3 + b])
                         : "r"(src + 256u * b + 8u * (uint32_t)(4 * g + t)));
        }
      }
      const uint32_t ic = (uint32_t)grp + 4u * oi;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t it = 2u * ic + (uint32_t)h;
        const int slot = it % kTcSlots;
        ok = __all_sync(0xffffffffu, wait_slot_free(it));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_col = tmem_base + lane_field + slot * kTcACols;
        if (act_ptr) {
          uint32_t x[4];
          if (act8) {           // signed bytes already; 2 bit: even columns of 0-7, of 8-15, odd of 0-7, of 8-15
            if (BITS == 2) {
              x[0] = tc_prmt(lv[h].x, lv[h].y, 0x6420u); x[1] = tc_prmt(lv[h].z, lv[h].w, 0x6420u);
              x[2] = tc_prmt(lv[h].x, lv[h].y, 0x7531u); x[3] = tc_prmt(lv[h].z, lv[h].w, 0x7531u);
            } else {
              x[0] = lv[h].x; x[1] = lv[h].y; x[2] = lv[h].z; x[3] = lv[h].w;
            }
          } else {
            const uint32_t w0 = lv[h].x, w1 = lv[h].y;
            const uint32_t e0 = w0 & 0x0f0f0f0fu, o0 = (w0 >> 4) & 0x0f0f0f0fu;
            const uint32_t e1 = w1 & 0x0f0f0f0fu, o1 = (w1 >> 4) & 0x0f0f0f0fu;
            if (BITS == 2) {    // lookup order of 16 columns: even fields of word 0, of word 1, odd fields of 0, of 1
              x[0] = e0; x[1] = e1; x[2] = o0; x[3] = o1;
            } else {            // natural order
              x[0] = tc_prmt(e0, o0, 0x5140u); x[1] = tc_prmt(e0, o0, 0x7362u);
              x[2] = tc_prmt(e1, o1, 0x5140u); x[3] = tc_prmt(e1, o1, 0x7362u);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) x[i] = ((x[i] | 0x80808080u) - 0x08080808u) ^ 0x80808080u;   // level - 8
          }
          uint8_t* row = gen_base + slot * kTcBBytes + (tk_token >> 3) * 1024 + (tk_token & 7) * 128;
          *reinterpret_cast<uint4*>(row + 16 * (tk_piece ^ (tk_token & 7))) = make_uint4(x[0], x[1], x[2], x[3]);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        // two quarters (64 weights) per store: a tcgen05.st costs about as much to issue whatever its width
#pragma unroll
        for (int tp = 0; tp < 2; ++tp) {
          uint32_t sel[16], v[16];
#pragma unroll
          for (int tq = 0; tq < 2; ++tq) {
            const int t = 2 * tp + tq;
            if (BITS == 2) {
#pragma unroll
              for (int wd = 0; wd < 2; ++wd) {
                const uint32_t r = raw[t][2 * h + wd];
                const uint32_t s0 = r & 0x33333333u, s1 = (r >> 2) & 0x33333333u;
                sel[8 * tq + 4 * wd] = s0; sel[8 * tq + 4 * wd + 1] = s0 >> 16;
                sel[8 * tq + 4 * wd + 2] = s1; sel[8 * tq + 4 * wd + 3] = s1 >> 16;
              }
            } else {
              const uint32_t r0 = raw[t][3 * h], r1 = raw[t][3 * h + 1], r2 = raw[t][3 * h + 2];
              const uint32_t ex = (((r0 >> 3) & 0x11111111u) | ((r1 >> 2) & 0x22222222u)) | ((r2 >> 1) & 0x44444444u);
              const uint32_t d0 = r0 & 0x77777777u, d1 = r1 & 0x77777777u, d2 = r2 & 0x77777777u;
              sel[8 * tq] = d0; sel[8 * tq + 1] = d0 >> 16; sel[8 * tq + 2] = d1; sel[8 * tq + 3] = d1 >> 16;
              sel[8 * tq + 4] = d2; sel[8 * tq + 5] = d2 >> 16; sel[8 * tq + 6] = ex; sel[8 * tq + 7] = ex >> 16;
            }
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = tc_prmt(TH[0], TH[1], sel[i]);
          tc_st16(a_col + 16 * tp, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = tc_prmt(TL[0], TL[1], sel[i]);
          tc_st16(a_col + 32 + 16 * tp, v);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        tc_arrive(full(slot));
      }
      __syncwarp();
      if (lane == 0 && fetched < n_own) { fetch(fetched); advance4(wf); ++fetched; }
      advance4(wc);
    }
    // copies still in flight must land before the CTA's shared memory is released
    if (lane == 0)
      for (uint32_t oi = consumed; oi < fetched; ++oi) tc_drain(ring_bar(dw, (int)(oi % kTcRing)), (oi / kTcRing) & 1u);
    __syncwarp();
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kTcFirstIssuer) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, (int)LCD_ERR_TIMEOUT);
}

template <int BITS>
size_t tc_smem_bytes() {
  return 1024 + (size_t)kTcSlots * kTcBBytes + (size_t)kTcDecoders * kTcRing * 2 * (512 * BITS) +
         8 * (3 * kTcSlots + 5 + kTcDecoders * kTcRing) + 16;
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

int tc_sm_count() { return current_sm_count(); }

// scratch of one problem: integer sums [n_rt][2][16][128], then tickets [n_rt][4]
struct TcScratch {
  size_t acc_off, ticket_off, end;
};
TcScratch tc_scratch(size_t begin, int64_t n_rt) {
  TcScratch s;
  s.acc_off = begin;
  s.ticket_off = s.acc_off + (size_t)n_rt * 2 * kTcTokens * kTcRows * sizeof(int);
  s.end = align256(s.ticket_off + (size_t)n_rt * 4 * sizeof(int));
  return s;
}

template <int BITS>
lcd_status tc_launch_t(const TcBatch& batch, int grid, int32_t* status, cudaStream_t stream) {
  auto kern = lut_gemv_tc_kernel<BITS>;
  const size_t smem = tc_smem_bytes<BITS>();
  static PerDeviceFlag attr_set;   // per template instance and device
  int dev;
  if (attr_set.first(&dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    attr_set.done(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  // weights are streamed before griddepcontrol.wait; levels, scales and scratch are touched after it
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, batch, status);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace

size_t lut_gemv_tc_workspace_bytes(const Problem* probs, int count) {
  size_t off = 0;
  for (int i = 0; i < count; ++i) off = tc_scratch(off, (probs[i].N_pad + kTcRows - 1) / kTcRows).end;
  return off;
}

lcd_status launch_lut_gemv_tc(const Problem* probs, int count, void* workspace, size_t workspace_bytes,
                              int32_t* status_word, void* stream) {
  if (count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  if (workspace_bytes < lut_gemv_tc_workspace_bytes(probs, count)) return LCD_ERR_BUFFER_TOO_SMALL;
  if (workspace == nullptr) return LCD_ERR_INVALID_ARG;
  const int bits = probs[0].bits;
  if (bits != 2 && bits != 3) return LCD_ERR_UNSUPPORTED;
  TcBatch batch;
  batch.count = count;
  size_t off = 0;
  unsigned long long total = 0;
  for (int i = 0; i < count; ++i) {
    const Problem& p = probs[i];
    if (p.bits != bits) return LCD_ERR_INVALID_ARG;
    if (p.M < 1 || p.M > kTcTokens) return LCD_ERR_UNSUPPORTED;
    TcProblem& g = batch.p[i];
    g.items = p.tiles;
    g.codebook = p.codebook;
    g.act_idx = p.act_idx;
    g.act_bits = p.act_bits;
    g.act_scale = p.act_scale;
    g.y = p.y;
    g.ldy = p.ldy;
    g.N = (int)p.N;
    g.M = (int)p.M;
    g.n_rp = (int)(p.N_pad / kPairRows);
    g.n_kt = (int)(p.K_pad / kTileK);
    g.n_rt = (int)((p.N_pad + kTcRows - 1) / kTcRows);
    g.unit0 = (unsigned)total;
    total += (unsigned long long)g.n_rt * (unsigned long long)g.n_kt;
    if (total > (1ull << 30)) return LCD_ERR_UNSUPPORTED;
    const TcScratch sl = tc_scratch(off, g.n_rt);
    g.acc = reinterpret_cast<int*>(static_cast<uint8_t*>(workspace) + sl.acc_off);
    g.ticket = reinterpret_cast<int*>(static_cast<uint8_t*>(workspace) + sl.ticket_off);
    off = sl.end;
  }
  for (int i = count; i < LCD_MAX_BATCH; ++i) batch.p[i] = batch.p[0];
  batch.total_units = (unsigned)total;
  const int n_sm = tc_sm_count();
  const int grid = total < (unsigned long long)n_sm ? (int)total : n_sm;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return bits == 2 ? tc_launch_t<2>(batch, grid, status_word, s) : tc_launch_t<3>(batch, grid, status_word, s);
}

}  // namespace lcd
