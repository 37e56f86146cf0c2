// Batched-prefill path (many tokens): the layer is a dense contraction y[M x N] = diag(s_q) * Q[M x K] * Wd[N x K]^T,
// where Wd[n][k] = cb[n][idx[n][k]] is what the lookup of Section 4.2 of the LCD paper returns and Q holds the
// activation levels of Section 4.1.  Two kernels share one structure (one persistent CTA per SM, tiles of 128 weight
// rows x BN tokens, every role a warp or a group of warps, mbarrier pipelines, accumulators in tensor memory):
//   dense_i8_kernel  (LCD_ALGO_DENSE_TC, the default)  int8 byte-table planes x int8 levels, kind::i8, int32 sums
//   dense_tc_kernel  (LCD_ALGO_DENSE_F16)              fp16 centroids x fp16 levels, kind::f16, fp32 sums
// Roles of dense_tc_kernel:
//   warp 0      TMA producer: token tiles (levels expanded once per call into the workspace, in the column order in
//               which the decoder emits weights) -> shared memory, 128-byte swizzle
//   warp 1      owns tensor memory; one lane issues tcgen05.mma (A and B from shared memory, two accumulator
//               buffers so that the epilogue overlaps the next tile)
//   warps 2-5   epilogue: tcgen05.ld, multiply by the token scale, coalesced fp32 stores
//   warps 6-21  decoder, two groups of 8 warps on alternate stages: packed 2/3-bit indices -> PRMT lookups in the
//               row's byte tables -> K-major 128-byte-swizzled A tile in shared memory
// Every wait is bounded (status word LCD_ERR_TIMEOUT on expiry, then every role leaves its loop, pending copies and
// MMAs are drained and tensor memory is released).
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "device_util.h"

namespace lcd {

namespace {

constexpr int kBM = 128;                 // weight rows per tile = MMA M
constexpr int kBK = 64;                  // columns per stage = one 128-byte swizzle row of fp16
constexpr int kStages = 4;
constexpr int kDecodeWarps = 16, kEpiWarps = 4;   // decoder: two groups of 8 warps
constexpr int kFirstEpiWarp = 2, kFirstDecodeWarp = kFirstEpiWarp + kEpiWarps;
constexpr int kDenseThreads = 32 * (kFirstDecodeWarp + kDecodeWarps);   // 704
constexpr int kABytes = kBM * kBK * 2;   // 16 KB per stage
constexpr unsigned long long kWaitNs = 2000000000ull;

__device__ __forceinline__ uint32_t prmt_b(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ unsigned long long timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void bar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when another role gave up (abort flag) or after kWaitNs, in which case the flag
// is raised for everybody.
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (bar_try(bar, parity)) return true;
  const unsigned long long t0 = timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (bar_try(bar, parity)) return true;
    if ((it & 255u) == 0) {
      if (*abort_flag) return false;
      if (timer_ns() - t0 > kWaitNs) { *abort_flag = 1; return false; }
    }
  }
}
// Wait used while draining after an abort: bounded by time only.
__device__ __forceinline__ void bar_drain(uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = timer_ns();
  for (uint32_t it = 1; !bar_try(bar, parity); ++it)
    if ((it & 255u) == 0 && timer_ns() - t0 > kWaitNs) return;
}

// 64-bit shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);       // start address
  d |= (uint64_t)(1024u >> 4) << 32;                      // stride byte offset
  d |= (uint64_t)1 << 46;                                 // descriptor version
  d |= (uint64_t)2 << 61;                                 // 128-byte swizzle
  return d;
}
// kind::f16 instruction descriptor: fp32 accumulate, fp16 A and B, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}

// ---------------------------------------------------------------------------------------------------------
// Activation levels as fp16, in the column order of the decoder.  One thread per (token, 32-column quarter):
// 16 bytes of packed 4-bit a = q + 8 in, 64 bytes of fp16 out.  Inside a quarter, position p holds column
//   3 bit: p;      2 bit: 16*(p>>4) + 8*((p>>2)&1) + 2*(p&3) + ((p>>3)&1)
// (the order in which the selector words of the 2-bit decoder list the weights).
template <int BITS>
__global__ void __launch_bounds__(256) expand_levels_kernel(const uint8_t* __restrict__ act_idx, int64_t n_quarters,
                                                            __half* __restrict__ out) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the tensor-core kernel may set itself up meanwhile
  const int64_t qi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (qi >= n_quarters) return;
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(act_idx) + qi);
  const uint32_t src[4] = {a.x, a.y, a.z, a.w};
  uint32_t o[16];
#pragma unroll
  for (int v = 0; v < 16; ++v) {
    uint32_t pair = 0;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int p = 2 * v + e;
      const int col = BITS != 2 ? p : 16 * (p >> 4) + 8 * ((p >> 2) & 1) + 2 * (p & 3) + ((p >> 3) & 1);
      const uint32_t nib = (src[col >> 3] >> (4 * (col & 7))) & 15u;
      pair |= (0x6400u | nib) << (16 * e);        // fp16 bits of 1024 + a
    }
    const __half2 h = __hsub2(*reinterpret_cast<const __half2*>(&pair), __floats2half2_rn(1032.0f, 1032.0f));   // a - 8, exact
    o[v] = *reinterpret_cast<const uint32_t*>(&h);
  }
  uint4* dst = reinterpret_cast<uint4*>(out + qi * 32);
#pragma unroll
  for (int c = 0; c < 4; ++c) dst[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
}

// ---------------------------------------------------------------------------------------------------------
struct DenseParams {
  const uint8_t* items;
  const uint16_t* codebook;
  const float* act_scale;
  float* y;
  long long ldy;
  int N, M, n_rp, n_kt, n_tiles_m, n_tiles;
  int32_t* status;
};

template <int BITS, int BN>
__global__ void __launch_bounds__(kDenseThreads, 1)
dense_tc_kernel(const __grid_constant__ CUtensorMap tmap_act, const DenseParams P) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int ITEM = 512 * BITS, HALF = 256 * BITS;
  constexpr int kBBytes = BN * kBK * 2;
  constexpr uint32_t kTmemCols = 2 * BN <= 256 ? 256 : 512;   // a power of two that holds both accumulator buffers
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t raw_addr = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - raw_addr);
  const uint32_t a_base = base, b_base = base + kStages * kABytes, bar_base = b_base + kStages * kBBytes;
  // barriers: full_a[4] full_b[4] empty[4] tmem_full[2] tmem_empty[2] drain
  auto full_a = [&](int s) { return bar_base + 8u * s; };
  auto full_b = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto empty = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
  auto tmem_full = [&](int b) { return bar_base + 8u * (3 * kStages + b); };
  auto tmem_empty = [&](int b) { return bar_base + 8u * (3 * kStages + 2 + b); };
  const uint32_t drain_bar = bar_base + 8u * (3 * kStages + 4);
  uint8_t* gen_misc = gen_base + kStages * (kABytes + kBBytes) + 8 * (3 * kStages + 5);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(gen_misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_misc + 4);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      bar_init(full_a(s), (kDecodeWarps / 2) * 32);   // one decoder group fills a stage
      bar_init(full_b(s), 1);
      bar_init(empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      bar_init(tmem_full(b), 1);
      bar_init(tmem_empty(b), kEpiWarps * 32);
    }
    bar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  const int n_ks = P.n_kt * 4;     // stages per tile

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      // the fp16 levels are written by the kernel launched just before this one: wait for it here (the other
      // roles only touch data that was complete before that kernel started)
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % P.n_tiles_m) * BN;
        for (int ks = 0; ks < n_ks; ++ks, ++it) {
          const int slot = it % kStages;
          if (!bar_wait(empty(slot), ((it / kStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          bar_expect_tx(full_b(slot), kBBytes);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(b_base + slot * kBBytes), "l"(&tmap_act), "r"(ks * kBK), "r"(m0), "r"(full_b(slot)) : "memory");
        }
      }
      // nothing this thread issued may still be in flight when the CTA exits
      const uint32_t n_back = it < (uint32_t)kStages ? it : (uint32_t)kStages;
      for (uint32_t i = 1; i <= n_back; ++i) {
        const uint32_t j = it - i;
        bar_drain(full_b(j % kStages), (j / kStages) & 1u);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(BN);
      const uint64_t a_desc0 = smem_desc(a_base), b_desc0 = smem_desc(b_base);
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, ++tl) {
        const uint32_t buf = tl & 1u;
        if (!bar_wait(tmem_empty(buf), ((tl >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int ks = 0; ks < n_ks; ++ks, ++it) {
          const int slot = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!bar_wait(full_a(slot), ph, abort_flag) || !bar_wait(full_b(slot), ph, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          // descriptors differ only in the start-address field (units of 16 bytes): this one thread issues every
          // MMA of the CTA, so its instruction count per stage is kept small
          const uint64_t ad = a_desc0 + (uint64_t)((slot * kABytes) >> 4), bd = b_desc0 + (uint64_t)((slot * kBBytes) >> 4);
          mma_f16(d_tmem, ad, bd, idesc, (uint32_t)(ks != 0));
#pragma unroll
          for (int k = 1; k < kBK / 16; ++k) mma_f16(d_tmem, ad + 2 * k, bd + 2 * k, idesc, 1u);
          mma_commit(empty(slot));
        }
        if (ok) mma_commit(tmem_full(buf));
      }
      // all MMAs issued so far must have finished before tensor memory is released
      mma_commit(drain_bar);
      bar_drain(drain_bar, 0);
    }
    __syncwarp();
  } else if (warp < kFirstDecodeWarp) {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;                    // tensor-memory lanes [32*quad, +32) belong to this warp
    uint32_t tl = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, ++tl) {
      const uint32_t buf = tl & 1u;
      const int n = (tile / P.n_tiles_m) * kBM + 32 * quad + lane;
      const int m0 = (tile % P.n_tiles_m) * BN;
      ok = __all_sync(0xffffffffu, bar_wait(tmem_full(buf), (tl >> 1) & 1u, abort_flag));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(32 * quad) << 16) + buf * BN + 32 * c, v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        const int mc = m0 + 32 * c;
        const float my_scale = mc + lane < P.M ? __ldg(P.act_scale + mc + lane) : 0.0f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float s = __shfl_sync(0xffffffffu, my_scale, j);
          if (mc + j < P.M && n < P.N) P.y[(size_t)(mc + j) * P.ldy + n] = __uint_as_float(v[j]) * s;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      bar_arrive(tmem_empty(buf));
    }
  } else {
    // ------------------------------------------------------------------ decoder
    // Two groups of 8 warps take alternate stages (group = stage parity), so that one group's shared-memory
    // stores, proxy fence and barrier round trip overlap the other group's lookups.  Inside a group, warp dw
    // owns the tile's 16-row group dw and a thread owns 32 columns of one row per stage.
    const int grp = (warp - kFirstDecodeWarp) >> 3, dw = (warp - kFirstDecodeWarp) & 7;
    const int u = lane >> 4, g = (lane >> 1) & 7, tq = lane & 1;
    const uint32_t row_off = (uint32_t)((2 * dw + u) * 1024 + g * 128);
    const int rec_lane = 4 * g + tq + 2 * grp;     // the quarter of the row this thread decodes: tq + 2 * grp
    uint32_t it0 = 0;                              // stage number of the tile's first stage
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, it0 += (uint32_t)n_ks) {
      int rp = (tile / P.n_tiles_m) * (kBM / 16) + dw;
      rp = rp < P.n_rp ? rp : P.n_rp - 1;          // rows past the matrix repeat the last group; never stored
      // byte tables of this thread's row: low and high bytes of the fp16 centroids
      uint32_t TL[2], TH[2];
      {
        const uint16_t* cb = P.codebook + ((size_t)rp * 16 + 8 * u + g) * (1 << BITS);
        if (BITS == 2) {
          const uint2 c = __ldg(reinterpret_cast<const uint2*>(cb));
          TL[0] = TL[1] = prmt_b(c.x, c.y, 0x6420u);
          TH[0] = TH[1] = prmt_b(c.x, c.y, 0x7531u);
        } else {
          const uint4 c = __ldg(reinterpret_cast<const uint4*>(cb));
          TL[0] = prmt_b(c.x, c.y, 0x6420u); TH[0] = prmt_b(c.x, c.y, 0x7531u);
          TL[1] = prmt_b(c.z, c.w, 0x6420u); TH[1] = prmt_b(c.z, c.w, 0x7531u);
        }
      }
      const uint8_t* row_items = P.items + (size_t)rp * P.n_kt * ITEM + u * HALF;
      // packed indices of this thread's quarter for one 256-column item: both 128-column k-blocks
      uint32_t cur[BITS * 2], nxt[BITS * 2];
      auto load_item = [&](uint32_t (&dst)[BITS * 2], int kt) {
        const uint8_t* item = row_items + (size_t)kt * ITEM;
        if (BITS == 2) {
          const uint4 r = __ldg(reinterpret_cast<const uint4*>(item + 16 * rec_lane));
          dst[0] = r.x; dst[1] = r.y; dst[2] = r.z; dst[3] = r.w;
        } else {
#pragma unroll
          for (int b = 0; b < 3; ++b) {
            const uint2 r = __ldg(reinterpret_cast<const uint2*>(item + 256 * b + 8 * rec_lane));
            dst[b] = r.x; dst[3 + b] = r.y;       // [0..2]: k-block 0, [3..5]: k-block 1
          }
        }
      };
      load_item(cur, 0);
      for (int kt = 0; kt < P.n_kt && ok; ++kt) {
        if (kt + 1 < P.n_kt) load_item(nxt, kt + 1);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // stage 2h + grp of the item: k-block h, quarters 2 * grp and 2 * grp + 1
          const uint32_t it = it0 + 4u * (uint32_t)kt + 2u * h + grp;
          const int slot = it % kStages;
          if (!bar_wait(empty(slot), ((it / kStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          uint32_t sel[8];
          if (BITS == 2) {
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              const uint32_t wd = cur[2 * h + x];
              const uint32_t s0 = wd & 0x33333333u, s1 = (wd >> 2) & 0x33333333u;
              sel[4 * x] = s0; sel[4 * x + 1] = s0 >> 16; sel[4 * x + 2] = s1; sel[4 * x + 3] = s1 >> 16;
            }
          } else {
            const uint32_t r0 = cur[3 * h], r1 = cur[3 * h + 1], r2 = cur[3 * h + 2];
            const uint32_t ex = (((r0 >> 3) & 0x11111111u) | ((r1 >> 2) & 0x22222222u)) | ((r2 >> 1) & 0x44444444u);
            const uint32_t d0 = r0 & 0x77777777u, d1 = r1 & 0x77777777u, d2 = r2 & 0x77777777u;
            sel[0] = d0; sel[1] = d0 >> 16; sel[2] = d1; sel[3] = d1 >> 16;
            sel[4] = d2; sel[5] = d2 >> 16; sel[6] = ex; sel[7] = ex >> 16;
          }
          uint8_t* a_row = gen_base + slot * kABytes + row_off;
#pragma unroll
          for (int c = 0; c < 4; ++c) {            // 16-byte chunk c of this thread's 32 columns
            uint32_t o[4];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              const uint32_t lo = prmt_b(TL[0], TL[1], sel[2 * c + x]), hi = prmt_b(TH[0], TH[1], sel[2 * c + x]);
              o[2 * x] = prmt_b(lo, hi, 0x5140u);
              o[2 * x + 1] = prmt_b(lo, hi, 0x7362u);
            }
            const int chunk = (4 * tq + c) ^ g;    // 128-byte swizzle: chunk index xor (row mod 8)
            *reinterpret_cast<uint4*>(a_row + 16 * chunk) = make_uint4(o[0], o[1], o[2], o[3]);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> visible to the MMA
          bar_arrive(full_a(slot));
        }
#pragma unroll
        for (int x = 0; x < BITS * 2; ++x) cur[x] = nxt[x];
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && P.status) atomicExch(P.status, (int)LCD_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------------
// Integer variant (the default for many tokens).  The row codebook becomes the same two byte tables as in the
// M <= 16 kernel (16-bit fixed point: signed high byte, unsigned low byte), the decoder emits two int8 A planes
// with ONE lookup per plane and four weights (no fp16 interleave), the levels are int8, and every stage of 128
// columns is multiplied twice with tcgen05.mma kind::i8 (twice the fp16 rate) into two int32 accumulators:
//     y = s_q * 2^e_n * (256 * D_hi + D_lo).
// Against the fp16 kernels this halves the token bytes streamed from L2 per flop (what bounds them) and halves
// the decoder's work; the sums are exact integers, the only error is the 2^-16 table quantisation.
// Tensor memory: (D_hi, D_lo) x BN columns per accumulator buffer.  Warps as in dense_tc_kernel plus a second MMA
// issuer; the two decoder groups take the two 128-column k-blocks of every item.
constexpr int kI8BK = 128;                      // columns per stage = one 128-byte swizzle row of int8
constexpr int kI8PlaneBytes = kBM * kI8BK;      // 16 KB per plane and stage
// Tiles of 128 tokens have two accumulator buffers (the epilogue overlaps the next tile); 192 and 256 tokens have
// one, but their MMAs are long enough (96 / 128 cycles) to hide the issue latency of the two issuing threads.
__host__ __device__ constexpr int i8_stages(int bn) { return bn <= 192 ? 4 : 3; }   // stages that fit in 227 KB
// warps: 0 TMA, 1 MMA issuer (high plane), 2-9 epilogue, 10-25 decoder, 26 MMA issuer (low plane)
constexpr int kI8EpiWarps = 8;
constexpr int kI8FirstDecodeWarp = kFirstEpiWarp + kI8EpiWarps;
constexpr int kI8Threads = 32 * (kI8FirstDecodeWarp + kDecodeWarps + 1);   // 864

// kind::i8 instruction descriptor: int32 accumulate, B signed, A signed (high plane) or unsigned (low plane).
__host__ __device__ constexpr uint32_t instr_desc_i8(int n, bool a_signed) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}
__device__ __forceinline__ void mma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr) : "memory");
}

// Waits for the tensor-memory loads in flight.  The loaded registers are operands: nothing that reads them can be
// scheduled before the wait.
__device__ __forceinline__ void tmem_wait8(uint32_t (&a)[8], uint32_t (&b)[8]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7])
               :: "memory");
}

// Activation levels as int8 in the decoder's column order (see expand_levels_kernel): one thread per (token,
// 32-column quarter), 16 bytes in, 32 bytes out.
template <int BITS>
__global__ void __launch_bounds__(256) expand_levels_i8_kernel(const uint8_t* __restrict__ act_idx, int64_t n_quarters,
                                                               int8_t* __restrict__ out) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t qi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (qi >= n_quarters) return;
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(act_idx) + qi);
  const uint32_t src[4] = {a.x, a.y, a.z, a.w};
  uint32_t o[8];
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int p = 4 * v + e;
      const int col = BITS != 2 ? p : 16 * (p >> 4) + 8 * ((p >> 2) & 1) + 2 * (p & 3) + ((p >> 3) & 1);
      const uint32_t nib = (src[col >> 3] >> (4 * (col & 7))) & 15u;
      word |= ((nib - 8u) & 0xffu) << (8 * e);       // q = a - 8 as a signed byte
    }
    o[v] = word;
  }
  uint4* dst = reinterpret_cast<uint4*>(out + qi * 32);
  dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
  dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// 8-bit levels (signed bytes, natural column order) in the 2-bit decoder's column order; one thread per quarter.
__global__ void __launch_bounds__(256) permute_levels_i8_kernel(const uint8_t* __restrict__ act_q, int64_t n_quarters,
                                                                int8_t* __restrict__ out) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t qi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (qi >= n_quarters) return;
  const uint4 a0 = __ldg(reinterpret_cast<const uint4*>(act_q) + 2 * qi);
  const uint4 a1 = __ldg(reinterpret_cast<const uint4*>(act_q) + 2 * qi + 1);
  const uint32_t src[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
  uint32_t o[8];
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    uint32_t word = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int p = 4 * v + e;
      const int col = 16 * (p >> 4) + 8 * ((p >> 2) & 1) + 2 * (p & 3) + ((p >> 3) & 1);
      word |= ((src[col >> 2] >> (8 * (col & 3))) & 0xffu) << (8 * e);
    }
    o[v] = word;
  }
  uint4* dst = reinterpret_cast<uint4*>(out + qi * 32);
  dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
  dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// 2^(e-15) of a row: e is the exponent with max|centroid| < 2^e (the scale of the row's 16-bit fixed point).
template <int BITS>
__device__ __forceinline__ float row_exponent_scale(const uint16_t* cb_row, float* up) {
  float mx = 0.0f;
#pragma unroll
  for (int i = 0; i < (1 << BITS); ++i) mx = fmaxf(mx, fabsf(__half2float(__ushort_as_half(__ldg(cb_row + i)))));
  int ex = (int)((__float_as_uint(mx) >> 23) & 0xffu) - 126;
  ex = ex < -30 ? -30 : ex;
  if (up) *up = __uint_as_float((uint32_t)(15 - ex + 127) << 23);
  return __uint_as_float((uint32_t)(ex - 15 + 127) << 23);
}

template <int BITS, int BN>
__global__ void __launch_bounds__(kI8Threads, 1)
dense_i8_kernel(const __grid_constant__ CUtensorMap tmap_act, const DenseParams P) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int ITEM = 512 * BITS, HALF = 256 * BITS;
  constexpr int kI8BBytes = BN * kI8BK;
  constexpr int kStages = i8_stages(BN);                          // shadows the fp16 kernels' stage count
  constexpr int NBUF = BN <= 128 ? 2 : 1;                         // accumulator buffers of (D_hi, D_lo) x BN columns
  constexpr int kStageBytes = 2 * kI8PlaneBytes + kI8BBytes;      // A high plane | A low plane | tokens
  constexpr uint32_t kTmemCols = 512;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t raw_addr = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - raw_addr);
  const uint32_t bar_base = base + kStages * kStageBytes;
  // full(s): the stage's operands are ready = all arrivals of one decoder group + the TMA producer's arrival
  // with its byte count
  auto full_a = [&](int s) { return bar_base + 8u * s; };
  auto full_b = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
  auto tmem_full = [&](int b) { return bar_base + 8u * (3 * kStages + b); };
  auto tmem_empty = [&](int b) { return bar_base + 8u * (3 * kStages + 2 + b); };
  const uint32_t drain_bar = bar_base + 8u * (3 * kStages + 4);
  uint8_t* gen_misc = gen_base + kStages * kStageBytes + 8 * (3 * kStages + 5);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(gen_misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_misc + 4);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      bar_init(full_a(s), (kDecodeWarps / 2) * 32 + 1);
      bar_init(empty(s), 2);                        // both MMA issuers release a stage
    }
    for (int b = 0; b < 2; ++b) {
      bar_init(tmem_full(b), 2);
      bar_init(tmem_empty(b), kI8EpiWarps * 32);
    }
    bar_init(drain_bar, 2);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  const int n_ks = P.n_kt * 2;     // stages per tile: the two 128-column k-blocks of every item

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (int8 levels)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % P.n_tiles_m) * BN;
        for (int ks = 0; ks < n_ks; ++ks, ++it) {
          const int slot = it % kStages;
          if (!bar_wait(empty(slot), ((it / kStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          bar_expect_tx(full_b(slot), kI8BBytes);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(base + slot * kStageBytes + 2 * kI8PlaneBytes), "l"(&tmap_act), "r"(ks * kI8BK), "r"(m0),
                "r"(full_b(slot)) : "memory");
        }
      }
      const uint32_t n_back = it < (uint32_t)kStages ? it : (uint32_t)kStages;
      for (uint32_t i = 1; i <= n_back; ++i) {
        const uint32_t j = it - i;
        bar_drain(full_b(j % kStages), (j / kStages) & 1u);
      }
    }
    __syncwarp();
  } else if (warp == 1 || warp == kI8Threads / 32 - 1) {
    // ------------------------------------------------------------------ MMA issuers
    // Two threads in two warps, one per byte plane (independent accumulators): a single thread cannot issue the
    // eight MMAs of a stage as fast as the tensor pipe executes them.
    if (lane == 0) {
      const bool is_hi = warp == 1;
      const uint32_t idesc = is_hi ? instr_desc_i8(BN, true) : instr_desc_i8(BN, false);
      const uint64_t desc0 = smem_desc(base) + (uint64_t)(is_hi ? 0 : (kI8PlaneBytes >> 4));
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, ++tl) {
        const uint32_t buf = tl % NBUF;
        if (!bar_wait(tmem_empty(buf), ((tl / NBUF) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d = tmem_base + buf * (2 * BN) + (is_hi ? 0 : BN);
        for (int ks = 0; ks < n_ks; ++ks, ++it) {
          const int slot = it % kStages;
          if (!bar_wait(full_a(slot), (it / kStages) & 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t ad = desc0 + (uint64_t)((slot * kStageBytes) >> 4);
          const uint64_t bd = smem_desc(base) + (uint64_t)((slot * kStageBytes + 2 * kI8PlaneBytes) >> 4);
          mma_i8(d, ad, bd, idesc, (uint32_t)(ks != 0));
#pragma unroll
          for (int k = 1; k < kI8BK / 32; ++k) mma_i8(d, ad + 2 * k, bd + 2 * k, idesc, 1u);   // 32 bytes per MMA
          mma_commit(empty(slot));
        }
        if (ok) mma_commit(tmem_full(buf));
      }
      mma_commit(drain_bar);
      bar_drain(drain_bar, 0);
    }
    __syncwarp();
  } else if (warp < kI8FirstDecodeWarp) {
    // ------------------------------------------------------------------ epilogue
    // two warps per tensor-memory quadrant, each drains every other 16-token chunk
    const int quad = warp & 3, half = (warp - kFirstEpiWarp) >> 2;
    uint32_t tl = 0;
    bool ok = true;
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the token scales may come from the kernel before this one
    for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, ++tl) {
      const uint32_t buf = tl % NBUF;
      const int n = (tile / P.n_tiles_m) * kBM + 32 * quad + lane;
      const int m0 = (tile % P.n_tiles_m) * BN;
      // this thread's row: 2^(e-15) of its fixed-point tables (rows past the matrix are never stored)
      const int n_cb = n < P.n_rp * 16 ? n : P.n_rp * 16 - 1;
      const float row_scale = row_exponent_scale<BITS>(P.codebook + (size_t)n_cb * (1 << BITS), nullptr);
      // The token scales of a pair of this warp's chunks live in one register: lane l holds the scale of token
      // l & 15 of chunk 2r + (l >> 4).  The first pair is asked for before the wait for the accumulators, the next
      // one while the current pair is drained.  (The chunk loop is not unrolled: measured no faster unrolled.)
      constexpr int kMyChunks = BN / 16 / (kI8EpiWarps / 4);
      static_assert(kMyChunks % 2 == 0, "an even number of 16-token chunks per epilogue warp");
      auto pair_scales = [&](int r) {
        const int m = m0 + 16 * (half + (kI8EpiWarps / 4) * (2 * r + (lane >> 4))) + (lane & 15);
        return m < P.M ? __ldg(P.act_scale + m) : 0.0f;
      };
      float sc_cur = pair_scales(0), sc_next = 0.0f;
      ok = __all_sync(0xffffffffu, bar_wait(tmem_full(buf), (tl / NBUF) & 1u, abort_flag));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float* y_row = P.y + (size_t)(m0 + 16 * half) * P.ldy + n;
      const bool row_ok = n < P.N;
      // Eight tokens at a time (sixteen accumulator registers leave room to overlap the tokens' dependent chains), two
      // register sets: the loads of the next eight are in flight while these are converted and stored.
      const uint32_t t_tile = tmem_base + ((uint32_t)(32 * quad) << 16) + buf * (2 * BN) + 16 * half;
      uint32_t hiA[8], loA[8], hiB[8], loB[8];
      tmem_ld8(t_tile, hiA);
      tmem_ld8(t_tile + BN, loA);
      auto drain8 = [&](const uint32_t (&hi)[8], const uint32_t (&lo)[8], float sc, int src0, int m_first, float* y8) {
        float s[8], v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) s[j] = __shfl_sync(0xffffffffu, sc, src0 + j) * row_scale;
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (float)(int)hi[j] * 256.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (v[j] + (float)(int)lo[j]) * s[j];
        if (m_first + 8 <= P.M) {          // (uniform) all eight tokens are inside: no test per token
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (row_ok) y8[(size_t)j * P.ldy] = v[j];
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (m_first + j < P.M && row_ok) y8[(size_t)j * P.ldy] = v[j];
        }
      };
#pragma unroll 1
      for (int i = 0; i < kMyChunks; ++i) {
        if ((i & 1) == 0) {
          if (i) sc_cur = sc_next;
          if (i + 2 < kMyChunks) sc_next = pair_scales((i >> 1) + 1);
        }
        const uint32_t t_chunk = t_tile + 16 * (kI8EpiWarps / 4) * i;
        const int mc = m0 + 16 * (half + (kI8EpiWarps / 4) * i);
        tmem_wait8(hiA, loA);
        tmem_ld8(t_chunk + 8, hiB);
        tmem_ld8(t_chunk + 8 + BN, loB);
        drain8(hiA, loA, sc_cur, 16 * (i & 1), mc, y_row);
        tmem_wait8(hiB, loB);
        if (i + 1 < kMyChunks) {
          tmem_ld8(t_chunk + 16 * (kI8EpiWarps / 4), hiA);
          tmem_ld8(t_chunk + 16 * (kI8EpiWarps / 4) + BN, loA);
        }
        drain8(hiB, loB, sc_cur, 16 * (i & 1) + 8, mc + 8, y_row + (size_t)8 * P.ldy);
        y_row += (size_t)(16 * (kI8EpiWarps / 4)) * P.ldy;
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      bar_arrive(tmem_empty(buf));
    }
  } else {
    // ------------------------------------------------------------------ decoder
    // Group 0 decodes k-block 0 of every item, group 1 k-block 1 (stage number parity).  Warp dw owns the tile's
    // 16-row group dw; a thread owns 64 columns (quarters 2x and 2x + 1) of one row per stage.
    const int grp = (warp - kI8FirstDecodeWarp) >> 3, dw = (warp - kI8FirstDecodeWarp) & 7;
    const int u = lane >> 4, g = (lane >> 1) & 7, x = lane & 1;
    const uint32_t row_off = (uint32_t)((2 * dw + u) * 1024 + g * 128);
    uint32_t it0 = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < P.n_tiles && ok; tile += gridDim.x, it0 += (uint32_t)n_ks) {
      int rp = (tile / P.n_tiles_m) * (kBM / 16) + dw;
      rp = rp < P.n_rp ? rp : P.n_rp - 1;          // rows past the matrix repeat the last group; never stored
      // byte tables of this thread's row: 16-bit fixed point, high (signed) and low (unsigned) bytes
      uint32_t TH[4] = {0, 0, 0, 0}, TL[4] = {0, 0, 0, 0};     // entries 4i .. 4i + 3 in word i (4 bit: all four words)
      {
        const uint16_t* cb = P.codebook + ((size_t)rp * 16 + 8 * u + g) * (1 << BITS);
        float up;
        (void)row_exponent_scale<BITS>(cb, &up);
#pragma unroll
        for (int i = 0; i < (1 << BITS); ++i) {
          const int f = __float2int_rn(__half2float(__ushort_as_half(__ldg(cb + i))) * up);
          TH[i >> 2] |= ((uint32_t)(f >> 8) & 0xffu) << (8 * (i & 3));
          TL[i >> 2] |= ((uint32_t)f & 0xffu) << (8 * (i & 3));
        }
        if (BITS == 2) { TH[1] = TH[0]; TL[1] = TL[0]; }
      }
      const uint8_t* row_items = P.items + (size_t)rp * P.n_kt * ITEM + u * HALF;
      constexpr int NW = BITS == 2 ? 2 : BITS == 3 ? 3 : 4;      // index words of a quarter of one k-block
      uint32_t cur[2][NW], nxt[2][NW];      // [quarter][word]
      auto load_stage = [&](uint32_t (&dst)[2][NW], int kt) {
        const uint8_t* item = row_items + (size_t)kt * ITEM;
#pragma unroll
        for (int xq = 0; xq < 2; ++xq) {
          const int l = 4 * g + 2 * x + xq;
          if (BITS == 2) {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(item + 16 * l + 8 * grp));
            dst[xq][0] = w.x; dst[xq][1] = w.y;
          } else if (BITS == 4) {           // one 512-byte plane per k-block, 16 bytes per lane
            const uint4 w = __ldg(reinterpret_cast<const uint4*>(item + 512 * grp + 16 * l));
            dst[xq][0] = w.x; dst[xq][1] = w.y; dst[xq][NW > 2 ? 2 : 0] = w.z; dst[xq][NW > 3 ? 3 : 0] = w.w;
          } else {
#pragma unroll
            for (int b = 0; b < 3; ++b)
              dst[xq][b] = __ldg(reinterpret_cast<const uint32_t*>(item + 256 * b + 8 * l + 4 * grp));
          }
        }
      };
      load_stage(cur, 0);
      for (int kt = 0; kt < P.n_kt && ok; ++kt) {
        if (kt + 1 < P.n_kt) load_stage(nxt, kt + 1);
        const uint32_t it = it0 + 2u * (uint32_t)kt + (uint32_t)grp;
        const int slot = it % kStages;
        // look everything up first (registers), wait for the stage to be free only then: the wait for the MMAs
        // that last read this stage overlaps the lookups
        uint32_t hw[2][2][4], lw[2][2][4];          // [quarter][chunk][word]
#pragma unroll
        for (int xq = 0; xq < 2; ++xq) {
          uint32_t sel[8], pick[8] = {0, 0, 0, 0, 0, 0, 0, 0};
          if (BITS == 4) {                  // natural order; pick = byte choice between entries 0..7 and 8..15
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {
              const uint32_t raw = cur[xq][NW > 3 ? wd : 0];
              const uint32_t s7 = raw & 0x77777777u, pk = ((raw >> 1) & 0x44444444u) | 0x32103210u;
              sel[2 * wd] = s7; sel[2 * wd + 1] = s7 >> 16; pick[2 * wd] = pk; pick[2 * wd + 1] = pk >> 16;
            }
          } else if (BITS == 2) {
#pragma unroll
            for (int wd = 0; wd < 2; ++wd) {
              const uint32_t raw = cur[xq][wd];
              const uint32_t s0 = raw & 0x33333333u, s1 = (raw >> 2) & 0x33333333u;
              sel[4 * wd] = s0; sel[4 * wd + 1] = s0 >> 16; sel[4 * wd + 2] = s1; sel[4 * wd + 3] = s1 >> 16;
            }
          } else {
            const uint32_t r0 = cur[xq][0], r1 = cur[xq][1], r2 = cur[xq][2];
            const uint32_t ex = (((r0 >> 3) & 0x11111111u) | ((r1 >> 2) & 0x22222222u)) | ((r2 >> 1) & 0x44444444u);
            const uint32_t d0 = r0 & 0x77777777u, d1 = r1 & 0x77777777u, d2 = r2 & 0x77777777u;
            sel[0] = d0; sel[1] = d0 >> 16; sel[2] = d1; sel[3] = d1 >> 16;
            sel[4] = d2; sel[5] = d2 >> 16; sel[6] = ex; sel[7] = ex >> 16;
          }
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              if (BITS == 4) {
                hw[xq][c][i] = prmt_b(prmt_b(TH[0], TH[1], sel[4 * c + i]), prmt_b(TH[2], TH[3], sel[4 * c + i]), pick[4 * c + i]);
                lw[xq][c][i] = prmt_b(prmt_b(TL[0], TL[1], sel[4 * c + i]), prmt_b(TL[2], TL[3], sel[4 * c + i]), pick[4 * c + i]);
              } else {
                hw[xq][c][i] = prmt_b(TH[0], TH[1], sel[4 * c + i]);
                lw[xq][c][i] = prmt_b(TL[0], TL[1], sel[4 * c + i]);
              }
            }
        }
        if (!bar_wait(empty(slot), ((it / kStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        uint8_t* a_row = gen_base + slot * kStageBytes + row_off;
#pragma unroll
        for (int xq = 0; xq < 2; ++xq)
#pragma unroll
          for (int c = 0; c < 2; ++c) {            // 16-byte chunk = 16 weights = four lookups, per plane
            const int chunk = (4 * x + 2 * xq + c) ^ g;     // 128-byte swizzle
            *reinterpret_cast<uint4*>(a_row + 16 * chunk) = make_uint4(hw[xq][c][0], hw[xq][c][1], hw[xq][c][2], hw[xq][c][3]);
            *reinterpret_cast<uint4*>(a_row + kI8PlaneBytes + 16 * chunk) =
                make_uint4(lw[xq][c][0], lw[xq][c][1], lw[xq][c][2], lw[xq][c][3]);
          }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> visible to the MMA
        bar_arrive(full_a(slot));
#pragma unroll
        for (int xq = 0; xq < 2; ++xq)
#pragma unroll
          for (int b = 0; b < NW; ++b) cur[xq][b] = nxt[xq][b];
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && P.status) atomicExch(P.status, (int)LCD_ERR_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int dense_sm_count() { return current_sm_count(); }

template <int BITS, int BN>
lcd_status launch_dense_t(const Problem& p, __half* levels, int32_t* status_word, cudaStream_t stream) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return LCD_ERR_CUDA;
  CUtensorMap tmap;
  const cuuint64_t dims[2] = {(cuuint64_t)p.K_pad, (cuuint64_t)p.M};
  const cuuint64_t strides[1] = {(cuuint64_t)p.K_pad * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)BN};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, levels, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return LCD_ERR_CUDA;
  DenseParams dp;
  dp.items = p.tiles;
  dp.codebook = p.codebook;
  dp.act_scale = p.act_scale;
  dp.y = p.y;
  dp.ldy = p.ldy;
  dp.N = (int)p.N;
  dp.M = (int)p.M;
  dp.n_rp = (int)(p.N_pad / kPairRows);
  dp.n_kt = (int)(p.K_pad / kTileK);
  dp.n_tiles_m = (int)((p.M + BN - 1) / BN);
  dp.n_tiles = dp.n_tiles_m * (int)((p.N_pad + kBM - 1) / kBM);
  dp.status = status_word;
  const size_t smem = 1024 + (size_t)kStages * (kABytes + BN * kBK * 2) + 256;
  auto kern = dense_tc_kernel<BITS, BN>;
  static PerDeviceFlag attr_set;   // per template instance and device
  int dev;
  if (attr_set.first(&dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    attr_set.done(dev);
  }
  const int grid = dp.n_tiles < dense_sm_count() ? dp.n_tiles : dense_sm_count();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kDenseThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see the producer's griddepcontrol.wait
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmap, dp);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

template <int BITS, int BN>
lcd_status launch_dense_i8(const Problem& p, int8_t* levels, int32_t* status_word, cudaStream_t stream) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return LCD_ERR_CUDA;
  CUtensorMap tmap;
  const cuuint64_t dims[2] = {(cuuint64_t)p.K_pad, (cuuint64_t)p.M};
  const cuuint64_t strides[1] = {(cuuint64_t)p.K_pad};
  const cuuint32_t box[2] = {(cuuint32_t)kI8BK, (cuuint32_t)BN};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, levels, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return LCD_ERR_CUDA;
  DenseParams dp;
  dp.items = p.tiles;
  dp.codebook = p.codebook;
  dp.act_scale = p.act_scale;
  dp.y = p.y;
  dp.ldy = p.ldy;
  dp.N = (int)p.N;
  dp.M = (int)p.M;
  dp.n_rp = (int)(p.N_pad / kPairRows);
  dp.n_kt = (int)(p.K_pad / kTileK);
  dp.n_tiles_m = (int)((p.M + BN - 1) / BN);
  dp.n_tiles = dp.n_tiles_m * (int)((p.N_pad + kBM - 1) / kBM);
  dp.status = status_word;
  const size_t smem = 1024 + (size_t)i8_stages(BN) * (2 * kI8PlaneBytes + BN * kI8BK) + 256;
  auto kern = dense_i8_kernel<BITS, BN>;
  static PerDeviceFlag attr_set;   // per template instance and device
  int dev;
  if (attr_set.first(&dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    attr_set.done(dev);
  }
  const int grid = dp.n_tiles < dense_sm_count() ? dp.n_tiles : dense_sm_count();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kI8Threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmap, dp);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

// Tile widths of the int8 kernel: {tokens, cycles per 64 columns of a tile, cycles per tile that do not overlap
// (the epilogue of the widths with one accumulator buffer)}, measured on the LLaMA-13B shapes at about 1.7 GHz.
// The launcher takes the width with the smallest waves x (columns x stage + fixed).
struct TileShape { int bn, stage_clks, epilogue_clks; };
constexpr TileShape kShapes[3] = {{128, 425, 0}, {192, 400, 6500}, {256, 535, 7500}};

int pick_shape(int64_t M, int64_t N_pad, int64_t n_ks) {
  const int n_sm = dense_sm_count();
  int best = 0;
  int64_t best_cost = -1;
  for (int i = 0; i < 3; ++i) {
    const TileShape& t = kShapes[i];
    const int64_t tiles = ((N_pad + kBM - 1) / kBM) * ((M + t.bn - 1) / t.bn);
    const int64_t cost = ((tiles + n_sm - 1) / n_sm) * (n_ks * t.stage_clks + t.epilogue_clks);
    if (best_cost < 0 || cost < best_cost) { best = i; best_cost = cost; }
  }
  return best;
}

}  // namespace

size_t dense_tc_workspace_bytes(int64_t M, int64_t K_pad) { return (size_t)round_up_u64((uint64_t)M * K_pad * 2, 256); }

lcd_status launch_dense_tc(const Problem& p, bool fp16_operands, void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream) {
  if (!p.dense_levels && (!workspace || workspace_bytes < dense_tc_workspace_bytes(p.M, p.K_pad))) return LCD_ERR_BUFFER_TOO_SMALL;
  if (p.M > 0x7fffffffLL / 2 || p.N > 0x7fffffffLL / 2) return LCD_ERR_UNSUPPORTED;
  if (p.bits == 4 && fp16_operands) return LCD_ERR_UNSUPPORTED;    // 4-bit indices: the int8 kernel only
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t n_quarters = p.M * (p.K_pad / 32);
  const unsigned blocks = (unsigned)((n_quarters + 255) / 256);
  if (p.act_bits == 8 && fp16_operands) return LCD_ERR_UNSUPPORTED;
  if (!fp16_operands) {
    int8_t* levels = static_cast<int8_t*>(workspace);
    if (p.dense_levels) {
      // the input transformation of this call has already written the signed bytes in this kernel's order
      levels = const_cast<int8_t*>(reinterpret_cast<const int8_t*>(p.act_idx));
    } else if (p.act_bits == 8) {
      // signed bytes already: the 3-bit decoder's order is the natural one, the 2-bit one needs the permutation
      if (p.bits == 2) permute_levels_i8_kernel<<<blocks, 256, 0, s>>>(p.act_idx, n_quarters, levels);
      else levels = const_cast<int8_t*>(reinterpret_cast<const int8_t*>(p.act_idx));
    } else if (p.bits == 2) expand_levels_i8_kernel<2><<<blocks, 256, 0, s>>>(p.act_idx, n_quarters, levels);
    else expand_levels_i8_kernel<3><<<blocks, 256, 0, s>>>(p.act_idx, n_quarters, levels);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    const int bn = kShapes[pick_shape(p.M, p.N_pad, p.K_pad / kBK)].bn;
    if (p.bits == 2) return bn == 128 ? launch_dense_i8<2, 128>(p, levels, status_word, s)
                          : bn == 192 ? launch_dense_i8<2, 192>(p, levels, status_word, s)
                                      : launch_dense_i8<2, 256>(p, levels, status_word, s);
    if (p.bits == 4) return bn == 128 ? launch_dense_i8<4, 128>(p, levels, status_word, s)
                          : bn == 192 ? launch_dense_i8<4, 192>(p, levels, status_word, s)
                                      : launch_dense_i8<4, 256>(p, levels, status_word, s);
    return bn == 128 ? launch_dense_i8<3, 128>(p, levels, status_word, s)
         : bn == 192 ? launch_dense_i8<3, 192>(p, levels, status_word, s)
                     : launch_dense_i8<3, 256>(p, levels, status_word, s);
  }
  __half* levels = static_cast<__half*>(workspace);
  if (p.bits == 2) expand_levels_kernel<2><<<blocks, 256, 0, s>>>(p.act_idx, n_quarters, levels);
  else expand_levels_kernel<3><<<blocks, 256, 0, s>>>(p.act_idx, n_quarters, levels);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  // 256-token tiles unless 128-token tiles need fewer waves per token
  const int n_sm = dense_sm_count();
  const int64_t tiles_n = (p.N_pad + kBM - 1) / kBM;
  const int64_t w256 = (tiles_n * ((p.M + 255) / 256) + n_sm - 1) / n_sm, w128 = (tiles_n * ((p.M + 127) / 128) + n_sm - 1) / n_sm;
  const bool wide = 2 * w256 <= w128;
  if (p.bits == 2) return wide ? launch_dense_t<2, 256>(p, levels, status_word, s) : launch_dense_t<2, 128>(p, levels, status_word, s);
  return wide ? launch_dense_t<3, 256>(p, levels, status_word, s) : launch_dense_t<3, 128>(p, levels, status_word, s);
}

}  // namespace lcd
