// LUT-GEMV for M <= 16 tokens (Section 4.2 of the LCD paper: values are fetched from a small per-row table by
// weight index and accumulated; no weight is dequantised to floating point and multiplied).
//
// Lookup.  Per output row the 2^bits centroids live in registers as byte tables; one PRMT instruction, whose
// selector nibbles are four weight indices, looks four weights up at once.  Two table sets exist:
//   kFixed16  - the fp16 centroids as 16-bit fixed point, a signed high-byte table and an unsigned low-byte
//               table; y = s_q * 2^e_n * (256 * sumH + sumL).
//   kBuckets  - Section 4.2, third paragraph (centroid-stationary buckets): one-hot tables, one per centroid
//               w >= 1, so that the accumulated value is the exact bucket sum S_w = sum_{k: idx = w} q_k;
//               S_0 is the token's sum of levels (an all-ones plane) minus the others, and
//               y = s_q * sum_w cb[w] * S_w in fp32: 2^bits multiplies per output.
// Accumulation.  The looked-up bytes are the A fragments of warp-level int8 tensor-core MMAs (m16n8k32), whose B
// fragments are the tokens' activation levels (int8, staged in shared memory in lookup order): 16 rows x 8
// tokens per instruction, exact int32 sums, so the result does not depend on the order of summation.
//
// Streaming.  The index area is a sequence of 16-row x 256-column items.  A run is one 16-row group x one column
// panel (a single panel when all tokens' levels of a whole row fit in shared memory).  A CTA owns whole runs, its
// 16 warps split the items of those runs evenly, and each warp streams its share through its own shared-memory
// ring filled by bulk asynchronous copies (cp.async.bulk + mbarrier), so many kilobytes per warp are in flight
// without holding registers.
//
// Combine.  Warps of a CTA that share a run add their integer partial sums in shared-memory slots with an arrival
// counter; the last one converts to fp32 and writes y.  With several panels (and for the bucket tables) the
// totals of a 16-row group meet in zero-filled global scratch with integer atomics; the warp that arrives last
// (ticket counter) writes y and leaves the scratch zero again.
//
// Several independent problems (the projections of a decoder layer) can run in one launch: CTAs are handed to the
// problems one at a time, each to the problem whose most loaded CTA has the most items.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "device_util.h"

namespace lcd {

namespace {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
// ring slots per warp: three, or two where 16 tokens need the shared memory for their activation levels
// (4-bit indices: items are 2 KB, three slots per warp would not leave room for the activation windows)
__host__ __device__ constexpr int ring_depth(int mg, int bits) { return (mg == 2 || bits == 4) ? 2 : 3; }
constexpr int kMaxDepth = 3;
constexpr int kStageItems = 2;       // items per slot
constexpr int kBarBytes = 512;       // mbarriers: kWarps * kMaxDepth * 8 = 384 bytes, padded
constexpr int kMaxSmem = 227 * 1024;
constexpr unsigned long long kTimeoutNs = 2000000000ull;   // bounded wait on a bulk copy: 2 s

struct GemvProblem {
  const uint8_t* items;       // index area
  const uint16_t* codebook;   // [N_pad][2^bits]
  const uint8_t* act_idx;     // [M][K_pad/2] packed 4-bit levels + 8, or [M][K_pad] signed bytes
  int act_bits;               // 4 or 8; 16: quantise x here (Section 4.1, dynamic per-token scale)
  const __half* x;            // act_bits == 16: [M][ldx] fp16
  const float* inv_smooth;    // act_bits == 16: [K] or null
  long long ldx;
  int K;                      // columns of x
  int x_vec;                  // rows of x and inv_smooth allow 16-byte loads and K % 8 == 0
  const float* act_scale;     // [M]
  float* y;
  int* acc;                   // scratch: [n_rp][MG][planes][4][32] int32, zero on entry and on exit
  int* ticket;                // scratch: [n_rp] int32, zero on entry and on exit
  long long ldy;
  int N, n_rp, n_kt, M;
  int pw;                     // columns are walked in panels of pw items (pw == n_kt: a single panel)
  int n_panels;
  int cta0, n_cta;            // CTAs [cta0, cta0 + n_cta) of the grid work on this problem, n_cta <= runs
  int tstride;                // bytes between tokens inside a staged activation window
};

struct GemvBatch {
  int count;
  int first_cta[LCD_MAX_BATCH];   // p[i].cta0 once more, side by side: a CTA finds its problem from one line of the
                                  // parameter block (entries from `count` on are INT_MAX)
  GemvProblem p[LCD_MAX_BATCH];
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
__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the phase did not complete within kTimeoutNs.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 1023u) == 0 && globaltimer() - t0 > kTimeoutNs) return false;
  }
}

enum TableKind { kFixed16 = 0, kBuckets = 1 };

template <int BITS, int KIND>
struct Planes {
  static constexpr int value = KIND == kFixed16 ? 2 : (1 << BITS);
};

// Byte tables of one row.  kFixed16: plane 0 = high bytes (signed), plane 1 = low bytes (unsigned); entries
// w = 0..3 in lo[], 4..7 in hi[] (3 bit).  kBuckets: the tables are the same for every row (one-hot) and are
// generated on the fly, only the centroid values are kept.
template <int BITS, int KIND>
struct RowTables {
  uint32_t lo[KIND == kFixed16 ? 2 : 1], hi[KIND == kFixed16 ? 2 : 1];   // [plane]
  uint32_t lo2[KIND == kFixed16 ? 2 : 1], hi2[KIND == kFixed16 ? 2 : 1]; // 4 bit: entries 8..11 and 12..15
  float scale;                                                          // kFixed16: 2^(e-15)
  float c[KIND == kBuckets ? (1 << BITS) : 1];                           // kBuckets: centroid values
};

template <int BITS>
struct RawCodebook {
  uint32_t w[BITS == 2 ? 2 : BITS == 3 ? 4 : 8];
};

template <int BITS>
__device__ __forceinline__ RawCodebook<BITS> load_codebook(const uint16_t* cb_row) {
  RawCodebook<BITS> r;
  if (BITS == 2) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(cb_row));
    r.w[0] = v.x; r.w[1] = v.y;
  } else {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(cb_row));
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
    if (BITS == 4) {
      const uint4 u = __ldg(reinterpret_cast<const uint4*>(cb_row) + 1);
      r.w[BITS == 4 ? 4 : 0] = u.x; r.w[BITS == 4 ? 5 : 0] = u.y; r.w[BITS == 4 ? 6 : 0] = u.z; r.w[BITS == 4 ? 7 : 0] = u.w;
    }
  }
  return r;
}

template <int BITS, int KIND>
__device__ __forceinline__ RowTables<BITS, KIND> build_tables(const RawCodebook<BITS>& raw) {
  constexpr int C = 1 << BITS;
  float v[C];
#pragma unroll
  for (int i = 0; i < C / 2; ++i) {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.w[i]));
    v[2 * i] = a.x; v[2 * i + 1] = a.y;
  }
  RowTables<BITS, KIND> T;
  if (KIND == kBuckets) {
#pragma unroll
    for (int i = 0; i < C; ++i) T.c[i] = v[i];
    T.scale = 1.0f;
    T.lo[0] = T.hi[0] = T.lo2[0] = T.hi2[0] = 0;
  } else {
    float mx = 0.0f;
#pragma unroll
    for (int i = 0; i < C; ++i) mx = fmaxf(mx, fabsf(v[i]));
    // mx < 2^ex from the exponent field (fp16 inputs are normal as floats); ex >= -30 keeps both powers finite
    int ex = (int)((__float_as_uint(mx) >> 23) & 0xffu) - 126;
    ex = ex < -30 ? -30 : ex;
    const float up = __uint_as_float((uint32_t)(15 - ex + 127) << 23);   // 2^(15-ex): |v| * up < 32768
    T.scale = __uint_as_float((uint32_t)(ex - 15 + 127) << 23);          // 2^(ex-15)
    uint32_t hb[4] = {0, 0, 0, 0}, lb[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < C; ++i) {
      const int f = __float2int_rn(v[i] * up);
      hb[i >> 2] |= ((uint32_t)(f >> 8) & 0xffu) << (8 * (i & 3));
      lb[i >> 2] |= ((uint32_t)f & 0xffu) << (8 * (i & 3));
    }
    T.lo[0] = hb[0]; T.lo[1] = lb[0];
    if (BITS >= 3) { T.hi[0] = hb[1]; T.hi[1] = lb[1]; } else { T.hi[0] = hb[0]; T.hi[1] = lb[0]; }
    T.lo2[0] = hb[2]; T.lo2[1] = lb[2]; T.hi2[0] = hb[3]; T.hi2[1] = lb[3];
  }
  return T;
}

// Four weights (selector nibbles of sel, low 16 bits) looked up in plane p of a row's tables.  p is a constant
// after unrolling.  kBuckets: plane p < C - 1 is the one-hot table of centroid p + 1 (byte w is 1 iff
// w == p + 1), the last plane is all ones.
// 4 bit: sel holds the low three bits of four indices, pick the byte choice 0x3210 + 4 * (bit 3 of each index)
// between the looked-up entries 0..7 and 8..15.
template <int BITS, int KIND>
__device__ __forceinline__ uint32_t pick_lookup(const RowTables<BITS, KIND>& T, uint32_t sel, int p, uint32_t pick = 0) {
  if (KIND == kFixed16 && BITS == 4) return prmt(prmt(T.lo[p], T.hi[p], sel), prmt(T.lo2[p], T.hi2[p], sel), pick);
  if (KIND == kFixed16) return prmt(T.lo[p], T.hi[p], sel);
  if (p == (1 << BITS) - 1) return 0x01010101u;
  const int w = p + 1;
  const uint32_t t_lo = w < 4 ? (1u << (8 * w)) : 0u;
  const uint32_t t_hi = BITS == 2 ? t_lo : (w >= 4 ? (1u << (8 * (w - 4))) : 0u);
  return prmt(t_lo, t_hi, sel);
}

// Activation levels of `n_words` source words (8 columns each, packed 4-bit a = q + 8, even column in the low
// nibble) as signed bytes, ordered the way the lookups emit weights.  Per 32-column quarter (4 source words):
//   2 bit: staged words [E(w0) E(w1) O(w0) O(w1) E(w2) E(w3) O(w2) O(w3)], E/O = even/odd columns of a word;
//   3 bit: natural column order.
// With 8-bit levels a group of 8 columns is two source words of signed bytes and only the order changes.
// One source word (act8: a pair) of a token's levels into its place j of the staged window.
template <int BITS>
__device__ __forceinline__ void stage_word(uint32_t* dst, int j, uint32_t a_lo, uint32_t a_hi, bool act8) {
  uint32_t e, o;
  if (act8) {
    if (BITS == 2) { e = prmt(a_lo, a_hi, 0x6420u); o = prmt(a_lo, a_hi, 0x7531u); }
    else { e = a_lo; o = a_hi; }
  } else {
    e = a_lo & 0x0f0f0f0fu; o = (a_lo >> 4) & 0x0f0f0f0fu;
    e = (e + 0x78787878u) ^ 0x80808080u;   // per byte a - 8, no carry between bytes
    o = (o + 0x78787878u) ^ 0x80808080u;
  }
  const int quarter = j >> 2, w = j & 3;
  if (BITS == 2) {
    dst[quarter * 8 + (w & 1) + 4 * (w >> 1)] = e;
    dst[quarter * 8 + 2 + (w & 1) + 4 * (w >> 1)] = o;
  } else if (act8) {
    dst[quarter * 8 + 2 * w] = e;
    dst[quarter * 8 + 2 * w + 1] = o;
  } else {
    dst[quarter * 8 + 2 * w] = prmt(e, o, 0x5140u);
    dst[quarter * 8 + 2 * w + 1] = prmt(e, o, 0x7362u);
  }
}
// The windows of n_tok tokens.  src: the first token's levels of the window's columns, the next token's
// src_stride words on (act8: pairs of words); dst likewise, dst_stride bytes apart.  The loads of eight tokens are
// issued together: one after the other they would cost a trip to L2 per token.
template <int BITS>
__device__ __forceinline__ void stage_window(uint8_t* dst, int dst_stride, const uint32_t* src, size_t src_stride,
                                             int n_tok, int n_words, int tid, bool act8) {
  for (int j = tid; j < n_words; j += kThreads) {
#pragma unroll 1
    for (int m0 = 0; m0 < n_tok; m0 += 8) {
      uint32_t lo[8], hi[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        lo[u] = hi[u] = 0u;
        if (m0 + u < n_tok) {
          if (act8) {
            const uint2 a = __ldcg(reinterpret_cast<const uint2*>(src + (size_t)(m0 + u) * src_stride * 2) + j);
            lo[u] = a.x; hi[u] = a.y;
          } else {
            lo[u] = __ldcg(src + (size_t)(m0 + u) * src_stride + j);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (m0 + u < n_tok)
          stage_word<BITS>(reinterpret_cast<uint32_t*>(dst + (size_t)(m0 + u) * dst_stride), j, lo[u], hi[u], act8);
    }
  }
}

// Levels of the 8 columns of group j (t = x * inv_s given) into a staged window: clip(rint(t * r)) as signed bytes in
// the lookup order.
template <int BITS>
__device__ __forceinline__ void store_levels(uint32_t* dst, int j, const float (&tv)[8], float r) {
  uint32_t b[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float q = rintf(__fmul_rn(tv[i], r));
    q = fminf(fmaxf(q, -8.0f), 7.0f);
    b[i] = (uint32_t)(int)q & 0xffu;
  }
  const int quarter = j >> 2, w = j & 3;
  if (BITS == 2) {
    dst[quarter * 8 + (w & 1) + 4 * (w >> 1)] = b[0] | (b[2] << 8) | (b[4] << 16) | (b[6] << 24);
    dst[quarter * 8 + 2 + (w & 1) + 4 * (w >> 1)] = b[1] | (b[3] << 8) | (b[5] << 16) | (b[7] << 24);
  } else {
    dst[quarter * 8 + 2 * w] = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
    dst[quarter * 8 + 2 * w + 1] = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
  }
}

// The same window straight from the fp16 activations (input transformation of Section 4.1 fused into the lookup
// kernel): level = clip(rint((x * inv_s) * r)), r = 7 / A with A the token's max |x * inv_s| (found beforehand),
// every step one binary32 operation as in quantize.cu, so the levels are the ones that kernel would write.
// k0: first column of the window; columns >= K are level 0.
template <int BITS>
__device__ __forceinline__ void stage_window_from_x(uint32_t* dst, const __half* xr, const float* inv_smooth, int k0,
                                                    int K, bool vec, float r, int n_words, int tid) {
  for (int j = tid; j < n_words; j += kThreads) {
    const int k = k0 + 8 * j;
    float tv[8];
    if (vec && k < K) {
      const uint4 raw = *reinterpret_cast<const uint4*>(xr + k);
      const __half2* h = reinterpret_cast<const __half2*>(&raw);
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
        tv[2 * i] = __fmul_rn(v.x, f[2 * i]);
        tv[2 * i + 1] = __fmul_rn(v.y, f[2 * i + 1]);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        tv[i] = k + i < K ? __fmul_rn(__half2float(xr[k + i]), inv_smooth ? __ldg(inv_smooth + k + i) : 1.0f) : 0.0f;
    }
    store_levels<BITS>(dst, j, tv, r);
  }
}

// Position inside a problem's item sequence, walked panel by panel: all 16-row groups of the first pw item
// columns, then of the next pw, ...
struct Cursor {
  uint32_t x, pn, rp, kk, pw;
};
__device__ __forceinline__ void cursor_set(Cursor& c, uint32_t x, const GemvProblem& P) {
  const uint32_t panel_items = (uint32_t)P.n_rp * (uint32_t)P.pw;
  c.x = x;
  c.pn = P.n_panels == 1 ? 0u : x / panel_items;
  const uint32_t r = x - c.pn * panel_items;
  const int left = P.n_kt - (int)c.pn * P.pw;
  c.pw = (uint32_t)(left < P.pw ? (left > 0 ? left : 1) : P.pw);
  c.rp = r / c.pw;
  c.kk = r - c.rp * c.pw;
}
__device__ __forceinline__ void cursor_advance(Cursor& c, uint32_t n, const GemvProblem& P) {
  c.x += n;
  c.kk += n;
  if (c.kk == c.pw) {
    c.kk = 0;
    if (++c.rp == (uint32_t)P.n_rp) {
      c.rp = 0;
      ++c.pn;
      const int left = P.n_kt - (int)c.pn * P.pw;
      c.pw = (uint32_t)(left < P.pw ? (left > 0 ? left : 1) : P.pw);
    }
  }
}
// Even split of n items over w parts: first item of part i, and the part that owns item x.
__device__ __forceinline__ uint32_t part_begin(uint32_t i, uint32_t n, uint32_t w) {
  return w == (uint32_t)kWarps ? (i * n) >> 4 : i * n / w;      // the split over a CTA's 16 warps needs no division
}
static_assert(kWarps == 16, "part_begin shifts by log2(kWarps)");
__device__ __forceinline__ uint32_t part_of(uint32_t x, uint32_t n, uint32_t w) { return ((x + 1) * w + n - 1) / n - 1; }

// Runs.  A run is the items of one 16-row group inside one panel (pw consecutive items in memory); runs are
// numbered panel by panel.  CTA c of a problem owns the runs [c*R/C, (c+1)*R/C); its warps split the items of
// those runs evenly.
struct RunGeometry {
  uint32_t n_rp, n_kt, pw, n_panels, n_runs, n_cta, n_items;
  __device__ __forceinline__ uint32_t panel_width(uint32_t pn) const {
    const uint32_t left = n_kt - pn * pw;
    return left < pw ? left : pw;
  }
  // first item (panel-major numbering) of run r; r == n_runs gives the item count
  __device__ __forceinline__ uint32_t run_start(uint32_t r) const {
    if (r >= n_runs) return n_items;
    if (n_panels == 1) return r * pw;          // the common case without a division (they are on the launch's critical path)
    const uint32_t pn = r / n_rp, rp = r - pn * n_rp;
    return pn * n_rp * pw + rp * panel_width(pn);
  }
  // warps that work on run (pn, rp): how many, and the first one's index inside its CTA
  __device__ __forceinline__ uint32_t contributors(uint32_t pn, uint32_t rp, uint32_t* first) const {
    const uint32_t r = pn * n_rp + rp;
    const uint32_t c = part_of(r, n_runs, n_cta);
    const uint32_t x0 = run_start(part_begin(c, n_runs, n_cta)), x1 = run_start(part_begin(c + 1, n_runs, n_cta));
    const uint32_t items = x1 - x0, nw = items < (uint32_t)kWarps ? items : (uint32_t)kWarps;
    const uint32_t xs = run_start(r) - x0, xe = xs + panel_width(pn) - 1;
    const uint32_t wf = part_of(xs, items, nw), wl = part_of(xe, items, nw);
    if (first) *first = wf;
    return wl - wf + 1;
  }
};

// One 16-row x 256-column item: look every weight up in its row's tables and accumulate against the tokens'
// levels.  item: the item's bytes in shared memory; q[G]: this lane's levels of token group G for the item.
template <int BITS, int KIND, int MG>
__device__ __forceinline__ void process_item(const uint8_t* item, const uint8_t* const (&q)[MG],
                                             const RowTables<BITS, KIND>& Ta, const RowTables<BITS, KIND>& Tb,
                                             int (&acc)[MG][Planes<BITS, KIND>::value][4], int lane) {
  constexpr int HALF = 256 * BITS;
  constexpr int PL = Planes<BITS, KIND>::value;
  uint32_t raw_a[BITS * 2], raw_b[BITS * 2];
  if (BITS == 2) {
    const uint4 wa = *reinterpret_cast<const uint4*>(item + 16 * lane);
    const uint4 wb = *reinterpret_cast<const uint4*>(item + HALF + 16 * lane);
    raw_a[0] = wa.x; raw_a[1] = wa.y; raw_a[2] = wa.z; raw_a[3] = wa.w;
    raw_b[0] = wb.x; raw_b[1] = wb.y; raw_b[2] = wb.z; raw_b[3] = wb.w;
  } else if (BITS == 4) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {       // one 512-byte plane per k-block
      const uint4 wa = *reinterpret_cast<const uint4*>(item + 512 * h + 16 * lane);
      const uint4 wb = *reinterpret_cast<const uint4*>(item + HALF + 512 * h + 16 * lane);
      raw_a[(BITS == 4 ? 4 : 0) * h] = wa.x; raw_a[(BITS == 4 ? 4 : 0) * h + 1] = wa.y;
      raw_a[(BITS == 4 ? 4 : 0) * h + 2] = wa.z; raw_a[(BITS == 4 ? 4 : 0) * h + (BITS == 4 ? 3 : 0)] = wa.w;
      raw_b[(BITS == 4 ? 4 : 0) * h] = wb.x; raw_b[(BITS == 4 ? 4 : 0) * h + 1] = wb.y;
      raw_b[(BITS == 4 ? 4 : 0) * h + 2] = wb.z; raw_b[(BITS == 4 ? 4 : 0) * h + (BITS == 4 ? 3 : 0)] = wb.w;
    }
  } else {
#pragma unroll
    for (int b = 0; b < 3; ++b) {
      const uint2 va = *reinterpret_cast<const uint2*>(item + 256 * b + 8 * lane);
      const uint2 vb = *reinterpret_cast<const uint2*>(item + HALF + 256 * b + 8 * lane);
      raw_a[b] = va.x; raw_a[3 + b] = va.y;
      raw_b[b] = vb.x; raw_b[3 + b] = vb.y;
    }
  }
  uint4 qv[2][2][MG];     // [k-block][staged words 0..3 / 4..7][token group]
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int G = 0; G < MG; ++G) {
      qv[h][0][G] = *reinterpret_cast<const uint4*>(q[G] + h * 128);
      qv[h][1][G] = *reinterpret_cast<const uint4*>(q[G] + h * 128 + 16);
    }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    uint32_t sel_a[8], sel_b[8];    // selector words of rows g and g + 8: lookup l uses the low 16 bits of sel[l]
    uint32_t pick_a[8] = {0, 0, 0, 0, 0, 0, 0, 0}, pick_b[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (BITS == 4) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {     // word w: eight indices in natural order
        const uint32_t ua = raw_a[(BITS == 4 ? 4 : 0) * h + (BITS == 4 ? w : 0)], ub = raw_b[(BITS == 4 ? 4 : 0) * h + (BITS == 4 ? w : 0)];
        const uint32_t a7 = ua & 0x77777777u, b7 = ub & 0x77777777u;
        const uint32_t ap = ((ua >> 1) & 0x44444444u) | 0x32103210u, bp = ((ub >> 1) & 0x44444444u) | 0x32103210u;
        sel_a[2 * w] = a7; sel_a[2 * w + 1] = a7 >> 16; pick_a[2 * w] = ap; pick_a[2 * w + 1] = ap >> 16;
        sel_b[2 * w] = b7; sel_b[2 * w + 1] = b7 >> 16; pick_b[2 * w] = bp; pick_b[2 * w + 1] = bp >> 16;
      }
    } else if (BITS == 2) {
#pragma unroll
      for (int w = 0; w < 2; ++w) {
        const uint32_t ua = raw_a[2 * h + w], ub = raw_b[2 * h + w];
        const uint32_t a0 = ua & 0x33333333u, a1 = (ua >> 2) & 0x33333333u;
        const uint32_t b0 = ub & 0x33333333u, b1 = (ub >> 2) & 0x33333333u;
        sel_a[4 * w] = a0; sel_a[4 * w + 1] = a0 >> 16; sel_a[4 * w + 2] = a1; sel_a[4 * w + 3] = a1 >> 16;
        sel_b[4 * w] = b0; sel_b[4 * w + 1] = b0 >> 16; sel_b[4 * w + 2] = b1; sel_b[4 * w + 3] = b1 >> 16;
      }
    } else {
      const uint32_t* ra = raw_a + 3 * h;
      const uint32_t* rb = raw_b + 3 * h;
      // bit b of columns 24..31 sits at bit 3 of the nibbles of word b: gather them into nibbles
      const uint32_t xa = (((ra[0] >> 3) & 0x11111111u) | ((ra[1] >> 2) & 0x22222222u)) | ((ra[2] >> 1) & 0x44444444u);
      const uint32_t xb = (((rb[0] >> 3) & 0x11111111u) | ((rb[1] >> 2) & 0x22222222u)) | ((rb[2] >> 1) & 0x44444444u);
#pragma unroll
      for (int b = 0; b < 3; ++b) {
        const uint32_t da = ra[b] & 0x77777777u, db = rb[b] & 0x77777777u;
        sel_a[2 * b] = da; sel_a[2 * b + 1] = da >> 16;
        sel_b[2 * b] = db; sel_b[2 * b + 1] = db >> 16;
      }
      sel_a[6] = xa; sel_a[7] = xa >> 16;
      sel_b[6] = xb; sel_b[7] = xb >> 16;
    }
    // four MMAs per plane: MMA j takes lookups 2j and 2j + 1 and staged words 2j, 2j + 1
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int p = 0; p < PL; ++p) {
        uint32_t a[4];
        a[0] = pick_lookup<BITS, KIND>(Ta, sel_a[2 * j], p, pick_a[2 * j]);
        a[1] = pick_lookup<BITS, KIND>(Tb, sel_b[2 * j], p, pick_b[2 * j]);
        a[2] = pick_lookup<BITS, KIND>(Ta, sel_a[2 * j + 1], p, pick_a[2 * j + 1]);
        a[3] = pick_lookup<BITS, KIND>(Tb, sel_b[2 * j + 1], p, pick_b[2 * j + 1]);
#pragma unroll
        for (int G = 0; G < MG; ++G) {
          const uint4& qq = qv[h][j >> 1][G];
          const uint32_t b0 = (j & 1) ? qq.z : qq.x, b1 = (j & 1) ? qq.w : qq.y;
          if (KIND == kFixed16 && p == 1) mma_u8(acc[G][p], a, b0, b1);
          else mma_s8(acc[G][p], a, b0, b1);
        }
      }
    }
  }
}

template <int BITS, int KIND, int MG>
__global__ void __launch_bounds__(kThreads, 1)
lut_gemv_kernel(const __grid_constant__ GemvBatch batch, int32_t* __restrict__ status) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int kDepth = ring_depth(MG, BITS);
  constexpr int ITEM = 512 * BITS;
  constexpr int SLOT = kStageItems * ITEM;
  constexpr int PL = Planes<BITS, KIND>::value;
  constexpr int ACC_INTS = MG * PL * 128;          // one warp's accumulators, [G][plane][reg][lane]
  constexpr bool kSmemCombine = KIND == kFixed16;  // partial sums of a CTA meet in shared memory
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;

  // which problem this CTA works on
  int pi = 0;
#pragma unroll
  for (int i = 1; i < LCD_MAX_BATCH; ++i) pi = (int)blockIdx.x >= batch.first_cta[i] ? i : pi;
  const GemvProblem& P = batch.p[pi];
  RunGeometry geo;
  geo.n_rp = (uint32_t)P.n_rp; geo.n_kt = (uint32_t)P.n_kt; geo.pw = (uint32_t)P.pw;
  geo.n_panels = (uint32_t)P.n_panels; geo.n_runs = geo.n_panels * geo.n_rp; geo.n_cta = (uint32_t)P.n_cta;
  geo.n_items = geo.n_rp * geo.n_kt;
  const uint32_t cta = blockIdx.x - P.cta0;
  // the CTA's items [cx0, cx1) in panel-major numbering and its warps' shares
  const uint32_t cx0 = geo.run_start(part_begin(cta, geo.n_runs, geo.n_cta));
  const uint32_t cx1 = geo.run_start(part_begin(cta + 1, geo.n_runs, geo.n_cta));
  const uint32_t c_items = cx1 - cx0;
  const uint32_t nw = c_items < (uint32_t)kWarps ? c_items : (uint32_t)kWarps;
  const bool warp_active = (uint32_t)warp < nw;
  const uint32_t wx0 = warp_active ? cx0 + part_begin(warp, c_items, nw) : cx0;
  const uint32_t wx1 = warp_active ? cx0 + part_begin(warp + 1, c_items, nw) : cx0;
  const uint32_t panel_items = geo.n_rp * geo.pw;
  const uint32_t pA = geo.n_panels == 1 ? 0u : cx0 / panel_items, pB = geo.n_panels == 1 ? 0u : (cx1 - 1) / panel_items;

  // shared memory: mbarriers | combine tickets | combine slots | rings | activation windows
  int* s_ticket = reinterpret_cast<int*>(smem + kBarBytes - 64);
  int* s_acc = reinterpret_cast<int*>(smem + kBarBytes);
  constexpr int COMBINE_BYTES = kSmemCombine ? kWarps * ACC_INTS * 4 : 0;
  uint8_t* ring = smem + kBarBytes + COMBINE_BYTES + (size_t)warp * kDepth * SLOT;
  const uint32_t bar0 = smem_u32(smem) + 8u * (uint32_t)(warp * kMaxDepth);
  uint8_t* act_s = smem + kBarBytes + COMBINE_BYTES + (size_t)kWarps * kDepth * SLOT;
  const int n_tok = P.M < 8 * MG ? P.M : 8 * MG;
  const int win_bytes = n_tok * P.tstride;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kDepth; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8u * s));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    s_ticket[warp] = 0;
  }
  __syncwarp();

  // Ring state.  Fetch side: next slot to fill, stages in flight, the rest of the segment being fetched (a
  // segment is this warp's share of one run: consecutive items in memory) and the cursor of the segment after
  // it.  Consumer side: next slot to read and its barrier phase.  Both sides cut every segment into stages of
  // kStageItems items from its start, so they agree on what each slot holds.
  uint32_t f_slot = 0, f_inflight = 0, f_left = 0, c_slot = 0, c_phase = 0;
  const uint8_t* f_src = P.items;
  const uint32_t ring_u32 = smem_u32(ring);
  bool aborted = false;
  Cursor fc = {0, 0, 0, 0, 1}, cc = fc;      // set for real before the first fetch (cursor_set below)

  uint64_t stream_policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
  auto issue_stage = [&]() {        // f_left > 0
    const uint32_t n = f_left < (uint32_t)kStageItems ? f_left : (uint32_t)kStageItems;
    if (lane == 0) {
      const uint32_t bar = bar0 + 8u * f_slot, bytes = n * ITEM, dst = ring_u32 + f_slot * SLOT;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      // weights are read once: evict-first keeps them from displacing what every CTA and every launch re-reads
      // (activations, smoothing factors, codebooks) from L2
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
          ::"r"(dst), "l"(f_src), "r"(bytes), "r"(bar), "l"(stream_policy) : "memory");
    }
    f_src += (size_t)n * ITEM;
    f_left -= n;
    f_slot = f_slot + 1 == (uint32_t)kDepth ? 0 : f_slot + 1;
    ++f_inflight;
  };
  // Issues the next stage if there is one before x_end.
  auto fetch_more = [&](uint32_t x_end) {
    if (f_left == 0) {
      if (fc.x >= x_end) return;
      const uint32_t row_left = fc.pw - fc.kk, range_left = x_end - fc.x;
      f_left = row_left < range_left ? row_left : range_left;
      f_src = P.items + ((size_t)fc.rp * P.n_kt + (size_t)fc.pn * P.pw + fc.kk) * ITEM;
      cursor_advance(fc, f_left, P);
    }
    issue_stage();
  };

  // The weights do not depend on the kernel that produced the activation indices: start streaming them (and
  // fetch the first rows' codebooks) before waiting for it.
  uint32_t round_lo, round_hi;
  {
    const uint32_t lo = pA * panel_items, hi = (pA + 2) * panel_items;
    round_lo = wx0 > lo ? wx0 : lo;
    round_hi = wx1 < hi ? wx1 : hi;
    if (round_hi < round_lo) round_hi = round_lo;
    cursor_set(fc, round_lo, P);
    cc = fc;
  }
  // Small loads first, bulk copies after them: an SM's loads return in the order they were queued, and a load
  // issued behind the ring's first fill waits for all of it (two microseconds for three stages of sixteen warps).
  RowTables<BITS, KIND> Ta, Tb;           // rows 16*rp + g and 16*rp + 8 + g
  RawCodebook<BITS> next_a, next_b;
  uint32_t tables_rp = 0xffffffffu, next_rp = cc.rp < geo.n_rp ? cc.rp : 0;
  next_a = load_codebook<BITS>(P.codebook + ((size_t)next_rp * 16 + g) * (1 << BITS));
  next_b = load_codebook<BITS>(P.codebook + ((size_t)next_rp * 16 + 8 + g) * (1 << BITS));
  // act_bits == 16, one token, one panel, at most kFastChunks * 4096 columns: the products x * inv_s stay in
  // registers between the maximum and the rounding, and the lines are asked into L2 before the dependency wait
  // (the weight stream evicts them between launches; a prefetch cannot read stale data, L2 is the coherence point)
  constexpr int kFastChunks = 3;
  const bool fused = P.act_bits == 16;
  const bool fast_stage = fused && P.x_vec && n_tok == 1 && P.n_panels == 1 && P.K <= kFastChunks * kThreads * 8;
  float fsm[kFastChunks][8];          // the smoothing factors do not depend on the previous kernel: read them now
  if (fast_stage) {
#pragma unroll
    for (int c = 0; c < kFastChunks; ++c) {
      const int k = (c * kThreads + tid) * 8;
#pragma unroll
      for (int i = 0; i < 8; ++i) fsm[c][i] = 1.0f;
      if (k < P.K) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(P.x + k));
        if (P.inv_smooth) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(P.inv_smooth + k));
          const float4 b = __ldg(reinterpret_cast<const float4*>(P.inv_smooth + k + 4));
          fsm[c][0] = a.x; fsm[c][1] = a.y; fsm[c][2] = a.z; fsm[c][3] = a.w;
          fsm[c][4] = b.x; fsm[c][5] = b.y; fsm[c][6] = b.z; fsm[c][7] = b.w;
        }
      }
    }
  }
  // Only one stage per warp is queued before the activations (or their stored levels) are asked for; the others
  // follow right behind that request.  The next kernel of the stream may be launched from here on (its blocks find
  // room as these finish; it waits for this grid's results itself).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  fetch_more(round_hi);
  bool ring_primed = false;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // the warp's combine slot is cleared here, with the first loads already under way (every use of it comes after
  // the block-wide barrier that ends the staging)
  if (kSmemCombine && !fast_stage)
    for (int i = lane; i < ACC_INTS; i += 32) s_acc[warp * ACC_INTS + i] = 0;

  // act_bits == 16: the tokens' maxima A = max_k |x_k * inv_s_k| first (each CTA for itself; x is a few KB in L2)
  float* s_amax = reinterpret_cast<float*>(smem + kWarps * kMaxDepth * 8);   // 16 floats between barriers and tickets
  if (fast_stage) {
    float* part = reinterpret_cast<float*>(act_s);
    uint4 xraw[kFastChunks];
#pragma unroll
    for (int c = 0; c < kFastChunks; ++c) {
      const int k = (c * kThreads + tid) * 8;
      xraw[c] = make_uint4(0u, 0u, 0u, 0u);
      if (k < P.K) xraw[c] = *reinterpret_cast<const uint4*>(P.x + k);
    }
    for (int i = 1; i < kDepth; ++i) fetch_more(round_hi);
    ring_primed = true;
    if (kSmemCombine)                        // cleared while the activations are on their way
      for (int i = lane; i < ACC_INTS; i += 32) s_acc[warp * ACC_INTS + i] = 0;
    float tv[kFastChunks][8];
    float amax = 0.0f;
#pragma unroll
    for (int c = 0; c < kFastChunks; ++c) {
      const int k = (c * kThreads + tid) * 8;
      if (k < P.K) {
        const __half2* h = reinterpret_cast<const __half2*>(&xraw[c]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __half22float2(h[i]);
          tv[c][2 * i] = __fmul_rn(v.x, fsm[c][2 * i]);
          tv[c][2 * i + 1] = __fmul_rn(v.y, fsm[c][2 * i + 1]);
          amax = fmaxf(amax, fmaxf(fabsf(tv[c][2 * i]), fabsf(tv[c][2 * i + 1])));
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) part[warp] = amax;
    __syncthreads();
    float A = 0.0f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) A = fmaxf(A, part[w]);
    if (tid == 0) s_amax[0] = A;
    __syncthreads();                                   // every thread has read the partial maxima: the window may be written
    const float r = A > 0.0f ? __fdiv_rn(7.0f, A) : 0.0f;
    uint32_t* dst = reinterpret_cast<uint32_t*>(act_s);
#pragma unroll
    for (int c = 0; c < kFastChunks; ++c) {
      const int k = (c * kThreads + tid) * 8;
      if (k < P.K) store_levels<BITS>(dst, k >> 3, tv[c], r);
    }
    const float zero[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    for (int j = (P.K >> 3) + tid; j < P.n_kt * 32; j += kThreads) store_levels<BITS>(dst, j, zero, 0.0f);   // padding columns
  } else if (fused) {
    float* part = reinterpret_cast<float*>(act_s);                            // [kWarps][16], before the windows exist
    for (int m = 0; m < n_tok; ++m) {
      const __half* xr = P.x + (size_t)m * P.ldx;
      float amax = 0.0f;
      if (P.x_vec) {
        for (int k = tid * 8; k < P.K; k += kThreads * 8) {
          const uint4 raw = *reinterpret_cast<const uint4*>(xr + k);
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
            amax = fmaxf(amax, fmaxf(fabsf(__fmul_rn(v.x, f[2 * i])), fabsf(__fmul_rn(v.y, f[2 * i + 1]))));
          }
        }
      } else {
        for (int k = tid; k < P.K; k += kThreads)
          amax = fmaxf(amax, fabsf(__fmul_rn(__half2float(xr[k]), P.inv_smooth ? __ldg(P.inv_smooth + k) : 1.0f)));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0) part[warp * 16 + m] = amax;
    }
    __syncthreads();
    if (tid < n_tok) {
      float v = 0.0f;
      for (int w = 0; w < kWarps; ++w) v = fmaxf(v, part[w * 16 + tid]);
      s_amax[tid] = v;
    }
    __syncthreads();
  }

  int acc[MG][PL][4];
#pragma unroll
  for (int G = 0; G < MG; ++G)
#pragma unroll
    for (int p = 0; p < PL; ++p)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[G][p][r] = 0;
  uint32_t seg_kk0 = 0;
  uint32_t tok_off[MG];
#pragma unroll
  for (int G = 0; G < MG; ++G) tok_off[G] = (uint32_t)((8 * G + g < P.M ? 8 * G + g : P.M - 1) * P.tstride + t * 32);

  // s_q of this lane's tokens 8G + 2t and 8G + 2t + 1 (asked for once: a load per output would put a trip to L2 into
  // every finished row group)
  float sq_tok[MG][2];
#pragma unroll
  for (int G = 0; G < MG; ++G)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int m = 8 * G + 2 * t + e;
      sq_tok[G][e] = 1.0f;
      if (m < P.M) {
        if (fused) {
          const float A = s_amax[m];
          sq_tok[G][e] = A > 0.0f ? __fdiv_rn(A, 7.0f) : 1.0f;
        } else {
          sq_tok[G][e] = __ldg(P.act_scale + m);
        }
      }
    }
  // y of the 16-row group rp from complete sums
  auto write_y = [&](uint32_t rp) {
#pragma unroll
    for (int G = 0; G < MG; ++G)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int m = 8 * G + 2 * t + (r & 1);
        const int n = 16 * (int)rp + g + ((r & 2) ? 8 : 0);
        if (m < P.M && n < P.N) {
          const RowTables<BITS, KIND>& T = (r & 2) ? Tb : Ta;
          float v;
          if (KIND == kFixed16) {
            v = T.scale * ((float)acc[G][0][r] * 256.0f + (float)acc[G][1][r]);
          } else {
            // planes 0..C-2 hold the exact bucket sums S_1..S_{C-1}, the last one the token's sum of levels
            int s0 = acc[G][PL - 1][r];
#pragma unroll
            for (int p = 0; p < PL - 1; ++p) s0 -= acc[G][p][r];
            v = T.c[0] * (float)s0;
#pragma unroll
            for (int p = 0; p < PL - 1; ++p) v = fmaf(T.c[p + 1], (float)acc[G][p][r], v);
          }
          P.y[(size_t)m * P.ldy + n] = v * sq_tok[G][r & 1];
        }
      }
  };
  // Adds this warp's sums to the global scratch of group rp; the warp that brings the count to `expected`
  // takes the totals back (leaving zeros) and writes y.
  auto global_combine = [&](uint32_t rp, uint32_t expected) {
    int* a = P.acc + (size_t)rp * ACC_INTS + lane;
#pragma unroll
    for (int G = 0; G < MG; ++G)
#pragma unroll
      for (int p = 0; p < PL; ++p)
#pragma unroll
        for (int r = 0; r < 4; ++r)
          if (8 * G + 2 * t + (r & 1) < P.M) atomicAdd(a + ((G * PL + p) * 4 + r) * 32, acc[G][p][r]);
    __threadfence();
    __syncwarp();
    int old = 0;
    if (lane == 0) old = atomicAdd(P.ticket + rp, 1);
    old = __shfl_sync(0xffffffffu, old, 0);
    if ((uint32_t)old + 1 == expected) {
      __threadfence();
#pragma unroll
      for (int G = 0; G < MG; ++G)
#pragma unroll
        for (int p = 0; p < PL; ++p)
#pragma unroll
          for (int r = 0; r < 4; ++r)
            if (8 * G + 2 * t + (r & 1) < P.M) acc[G][p][r] = atomicExch(a + ((G * PL + p) * 4 + r) * 32, 0);
      if (lane == 0) atomicExch(P.ticket + rp, 0);
      write_y(rp);
    }
  };
  // This warp's share [seg_kk0, kk_end) of run (pn, rp) is summed: combine it with the other warps' shares.
  auto flush = [&](uint32_t rp, uint32_t pn, uint32_t pw_n, uint32_t kk_end) {
    const bool whole = seg_kk0 == 0 && kk_end == pw_n;
    if (kSmemCombine) {
      bool run_done = whole;
      if (!whole) {
        uint32_t first = 0, n_contrib;
        if (nw == (uint32_t)kWarps) {
          // the run belongs to this CTA and this warp works on it: the other warps on it are its neighbours, found by
          // walking the warps' first items (shares are a CTA's items split evenly, see wx0) down and up from here
          const uint32_t xs = geo.run_start(pn * geo.n_rp + rp) - cx0, xe = xs + pw_n - 1;
          uint32_t wf = (uint32_t)warp, wl = (uint32_t)warp;
          while (wf > 0 && part_begin(wf, c_items, nw) > xs) --wf;
          while (wl + 1 < nw && part_begin(wl + 1, c_items, nw) <= xe) ++wl;
          first = wf;
          n_contrib = wl - wf + 1;
        } else {
          n_contrib = geo.contributors(pn, rp, &first);
        }
        int* a = s_acc + first * ACC_INTS + lane;
#pragma unroll
        for (int G = 0; G < MG; ++G)
#pragma unroll
          for (int p = 0; p < PL; ++p)
#pragma unroll
            for (int r = 0; r < 4; ++r) atomicAdd(a + ((G * PL + p) * 4 + r) * 32, acc[G][p][r]);
        __threadfence_block();
        __syncwarp();
        int old = 0;
        if (lane == 0) old = atomicAdd(s_ticket + first, 1);
        old = __shfl_sync(0xffffffffu, old, 0);
        run_done = (uint32_t)old + 1 == n_contrib;
        if (run_done) {
          __threadfence_block();
#pragma unroll
          for (int G = 0; G < MG; ++G)
#pragma unroll
            for (int p = 0; p < PL; ++p)
#pragma unroll
              for (int r = 0; r < 4; ++r)
                acc[G][p][r] = *reinterpret_cast<volatile int*>(a + ((G * PL + p) * 4 + r) * 32);
        }
      }
      if (run_done) {
        if (P.n_panels == 1) write_y(rp);
        else global_combine(rp, (uint32_t)P.n_panels);
      }
    } else {
      if (whole && P.n_panels == 1) {
        write_y(rp);
      } else {
        uint32_t part = 0;
        if (lane < P.n_panels) part = geo.contributors((uint32_t)lane, rp, nullptr);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        global_combine(rp, part);
      }
    }
#pragma unroll
    for (int G = 0; G < MG; ++G)
#pragma unroll
      for (int p = 0; p < PL; ++p)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[G][p][r] = 0;
  };

#pragma unroll 1
  for (uint32_t pbase = pA; pbase <= pB; pbase += 2) {
    if (pbase != pA) {
      const uint32_t lo = pbase * panel_items, hi = (pbase + 2) * panel_items;
      round_lo = wx0 > lo ? wx0 : lo;
      round_hi = wx1 < hi ? wx1 : hi;
      if (round_hi < round_lo) round_hi = round_lo;
      cursor_set(fc, round_lo, P);
      cc = fc;
      if (!aborted)
        for (int i = 0; i < kDepth; ++i) fetch_more(round_hi);
      __syncthreads();     // every warp is done with the previous windows
    }
    // stage the activation windows of panels pbase and pbase + 1
#pragma unroll 1
    for (uint32_t wdw = 0; wdw < 2 && pbase + wdw <= pB; ++wdw) {
      const uint32_t pn = pbase + wdw;
      const int n_words = (int)geo.panel_width(pn) * 32;
      if (fused) {
        for (int m = 0; m < n_tok && !fast_stage; ++m) {
          uint32_t* dst = reinterpret_cast<uint32_t*>(act_s + wdw * win_bytes + m * P.tstride);
          const float A = s_amax[m];
          stage_window_from_x<BITS>(dst, P.x + (size_t)m * P.ldx, P.inv_smooth, (int)(pn * P.pw) * 256, P.K,
                                    P.x_vec != 0, A > 0.0f ? __fdiv_rn(7.0f, A) : 0.0f, n_words, tid);
        }
      } else {
        const bool act8 = P.act_bits == 8;
        stage_window<BITS>(act_s + wdw * win_bytes, P.tstride,
                           reinterpret_cast<const uint32_t*>(P.act_idx + (size_t)pn * P.pw * 128 * (act8 ? 2 : 1)),
                           (size_t)P.n_kt * 32, n_tok, n_words, tid, act8);
      }
    }
    if (!ring_primed) {            // first pass: the staging loads above are queued, now the rest of the ring
      for (int i = 1; i < kDepth; ++i) fetch_more(round_hi);
      ring_primed = true;
    }
    __syncthreads();

    if (warp_active && !aborted) {
#pragma unroll 1
      while (cc.x < round_hi) {
        // one segment: this warp's share of run (cc.pn, cc.rp), seg_len consecutive items from column item cc.kk
        const uint32_t rp = cc.rp, pn = cc.pn, pw_n = cc.pw, kk0 = cc.kk;
        const uint32_t row_left = pw_n - kk0, range_left = round_hi - cc.x;
        const uint32_t seg_len = row_left < range_left ? row_left : range_left;
        // row tables of this 16-row group (its codebook rows were requested one group ahead)
        if (rp != tables_rp) {
          if (next_rp != rp) {
            next_a = load_codebook<BITS>(P.codebook + ((size_t)rp * 16 + g) * (1 << BITS));
            next_b = load_codebook<BITS>(P.codebook + ((size_t)rp * 16 + 8 + g) * (1 << BITS));
          }
          Ta = build_tables<BITS, KIND>(next_a);
          Tb = build_tables<BITS, KIND>(next_b);
          tables_rp = rp;
          next_rp = rp + 1 < geo.n_rp ? rp + 1 : 0;
          next_a = load_codebook<BITS>(P.codebook + ((size_t)next_rp * 16 + g) * (1 << BITS));
          next_b = load_codebook<BITS>(P.codebook + ((size_t)next_rp * 16 + 8 + g) * (1 << BITS));
        }
        const uint8_t* q[MG];
#pragma unroll
        for (int G = 0; G < MG; ++G) q[G] = act_s + (pn - pbase) * win_bytes + (size_t)kk0 * 256 + tok_off[G];
#pragma unroll 1
        for (uint32_t left = seg_len; left > 0;) {
          const uint32_t n = left < (uint32_t)kStageItems ? left : (uint32_t)kStageItems;
          const bool ok = __all_sync(0xffffffffu, mbar_wait(bar0 + 8u * c_slot, c_phase));
          if (!ok) { aborted = true; break; }
          const uint8_t* slot_p = ring + c_slot * SLOT;
          process_item<BITS, KIND, MG>(slot_p, q, Ta, Tb, acc, lane);
          if (kStageItems > 1 && n > 1) {
            const uint8_t* q1[MG];
#pragma unroll
            for (int G = 0; G < MG; ++G) q1[G] = q[G] + 256;
            process_item<BITS, KIND, MG>(slot_p + ITEM, q1, Ta, Tb, acc, lane);
          }
#pragma unroll
          for (int G = 0; G < MG; ++G) q[G] += n * 256;
          left -= n;
          __syncwarp();
          --f_inflight;
          if (++c_slot == (uint32_t)kDepth) { c_slot = 0; c_phase ^= 1u; }
          fetch_more(round_hi);                   // the slot just read is free again
        }
        if (aborted) {
          if (lane == 0 && status) atomicExch(status, (int)LCD_ERR_TIMEOUT);
          break;
        }
        cursor_advance(cc, seg_len, P);
        seg_kk0 = kk0;
        flush(rp, pn, pw_n, kk0 + seg_len);
      }
    }
    if (aborted) {
      // copies already issued must land before the CTA may exit
      while (f_inflight > 0) {
        (void)mbar_wait(bar0 + 8u * c_slot, c_phase);
        --f_inflight;
        if (++c_slot == (uint32_t)kDepth) { c_slot = 0; c_phase ^= 1u; }
      }
      f_left = 0;
    }
  }
}

}  // namespace

namespace {

int sm_count() { return current_sm_count(); }

// items (16 rows x 256 columns) of a launch from which LCD_ALGO_AUTO takes the shared-memory bucket tables.  Their
// launch costs about 7 us before and after the lookups (token maximum, tables, the grid-wide finish) against 3.5 us
// of the register tables, and looks weights up 1.6 times as fast: measured per launch, 4096 x 4096 7.3 vs 5.7 us,
// 11008 x 4096 9.3 vs 8.3, the seven matrices of a LLaMA-7B-shaped layer (49408 items) 20.0 vs 22.4, the three of a
// LLaMA-70B-shaped MLP 46 vs 59.
constexpr long long kSharedBucketMinItems = 32768;

int planes_of(int bits, int kind) { return kind == kFixed16 ? 2 : (1 << bits); }

struct ScratchLayout {
  size_t acc_off, ticket_off, end;
};
ScratchLayout scratch_layout(size_t begin, int64_t n_rp, int MG, int planes) {
  ScratchLayout s;
  s.acc_off = begin;
  s.ticket_off = s.acc_off + (size_t)n_rp * MG * planes * 128 * sizeof(int);
  s.end = (size_t)round_up_u64(s.ticket_off + (size_t)n_rp * sizeof(int), 256);
  return s;
}

template <int BITS, int KIND, int MG>
lcd_status launch_t(const GemvBatch& batch, int grid, size_t smem, int32_t* status, cudaStream_t stream) {
  auto kern = lut_gemv_kernel<BITS, KIND, MG>;
  static PerDeviceFlag attr_set;   // per template instance and device
  int dev;
  if (attr_set.first(&dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    attr_set.done(dev);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  // The kernel may start while the previous kernel of the stream drains: it streams weights first and waits
  // (griddepcontrol.wait) before it touches the activation indices.
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

// LCD_ALGO_AUTO for at most 16 tokens: the shared-memory bucket tables where they apply (one token, 2-bit indices)
// and the launch has enough rows per CTA to pay for building them, else the register tables.
lcd_algo resolve_small_m(const Problem* probs, int count, lcd_algo algo) {
  if (algo != LCD_ALGO_AUTO) return algo;
  if (!lut_smem_supported(probs, count)) return LCD_ALGO_REGISTER_LUT;
  long long items = 0;
  for (int i = 0; i < count; ++i) items += (probs[i].N_pad / kPairRows) * (probs[i].K_pad / kTileK);
  return items >= kSharedBucketMinItems ? LCD_ALGO_SHARED_BUCKET : LCD_ALGO_REGISTER_LUT;
}

size_t lut_gemv_workspace_bytes(const Problem* probs, int count, lcd_algo algo) {
  if (algo == LCD_ALGO_TC_LUT) return lut_gemv_tc_workspace_bytes(probs, count);
  if (algo == LCD_ALGO_SHARED_BUCKET) return lut_smem_workspace_bytes(probs, count);
  const int kind = algo == LCD_ALGO_BUCKET_LUT ? kBuckets : kFixed16;
  int64_t max_m = 1;
  for (int i = 0; i < count; ++i) max_m = probs[i].M > max_m ? probs[i].M : max_m;
  const int MG = max_m > 8 ? 2 : 1;
  size_t off = 0;
  for (int i = 0; i < count; ++i)
    off = scratch_layout(off, probs[i].N_pad / kPairRows, MG, planes_of(probs[i].bits, kind)).end;
  return off;
}

lcd_status launch_lut_gemv(const Problem* probs, int count, lcd_algo algo, void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream) {
  if (count < 1 || count > LCD_MAX_BATCH) return LCD_ERR_INVALID_ARG;
  if (algo == LCD_ALGO_TC_LUT) return launch_lut_gemv_tc(probs, count, workspace, workspace_bytes, status_word, stream);
  if (algo == LCD_ALGO_SHARED_BUCKET) return launch_lut_smem(probs, count, workspace, workspace_bytes, status_word, stream);
  const int kind = algo == LCD_ALGO_BUCKET_LUT ? kBuckets : kFixed16;
  const int bits = probs[0].bits;
  int64_t max_m = 1;
  for (int i = 0; i < count; ++i) {
    if (probs[i].bits != bits || probs[i].M > 16 || probs[i].M < 1) return LCD_ERR_UNSUPPORTED;
    max_m = probs[i].M > max_m ? probs[i].M : max_m;
  }
  const int MG = max_m > 8 ? 2 : 1;
  const int planes = planes_of(bits, kind);
  if (workspace_bytes < lut_gemv_workspace_bytes(probs, count, algo) || !workspace) return LCD_ERR_BUFFER_TOO_SMALL;

  const int item_bytes = 512 * bits;
  const size_t ring_bytes = (size_t)kWarps * ring_depth(MG, bits) * kStageItems * item_bytes;
  const size_t combine_bytes = kind == kFixed16 ? (size_t)kWarps * MG * planes * 128 * sizeof(int) : 0;
  const size_t act_budget = (size_t)kMaxSmem - kBarBytes - combine_bytes - ring_bytes;

  GemvBatch batch;
  batch.count = count;
  size_t act_bytes = 0, off = 0;
  for (int i = 0; i < count; ++i) {
    const Problem& p = probs[i];
    GemvProblem& g = batch.p[i];
    g.items = p.tiles;
    g.codebook = p.codebook;
    g.act_idx = p.act_idx;
    g.act_bits = p.act_bits;
    g.x = static_cast<const __half*>(p.x_fp16);
    g.inv_smooth = p.inv_smooth;
    g.ldx = p.ldx;
    g.K = (int)p.K;
    g.x_vec = (p.K % 8 == 0) && (p.ldx % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.x_fp16) & 15) == 0) &&
              (!p.inv_smooth || (reinterpret_cast<uintptr_t>(p.inv_smooth) & 15) == 0);
    g.act_scale = p.act_scale;
    g.y = p.y;
    g.ldy = p.ldy;
    g.N = (int)p.N;
    g.n_rp = (int)(p.N_pad / kPairRows);
    g.n_kt = (int)(p.K_pad / kTileK);
    g.M = (int)p.M;
    if ((int64_t)g.n_rp * g.n_kt > (1LL << 30) / 16) return LCD_ERR_UNSUPPORTED;
    const ScratchLayout sl = scratch_layout(off, g.n_rp, MG, planes);
    g.acc = reinterpret_cast<int*>(static_cast<uint8_t*>(workspace) + sl.acc_off);
    g.ticket = reinterpret_cast<int*>(static_cast<uint8_t*>(workspace) + sl.ticket_off);
    off = sl.end;
    // panels: a single one when all tokens' levels of the whole row fit, else the fewest that let two
    // panel windows fit
    const size_t m_eff = (size_t)(g.M < 8 * MG ? g.M : 8 * MG);
    int n_panels = 1, pw = g.n_kt;
    if (m_eff * ((size_t)g.n_kt * 256 + 16) > act_budget) {
      for (n_panels = 2;; ++n_panels) {
        pw = (g.n_kt + n_panels - 1) / n_panels;
        if (2 * m_eff * ((size_t)pw * 256 + 16) <= act_budget) break;
        if (pw == 1) return LCD_ERR_UNSUPPORTED;
      }
      n_panels = (g.n_kt + pw - 1) / pw;
      if (n_panels > 32) return LCD_ERR_UNSUPPORTED;
    }
    g.pw = pw;
    g.n_panels = n_panels;
    g.tstride = pw * 256 + 16;
    const size_t need = (n_panels == 1 ? 1 : 2) * m_eff * (size_t)g.tstride;
    act_bytes = need > act_bytes ? need : act_bytes;
    // act_bits == 16: the window area first holds the warps' partial maxima, kWarps x 16 floats
    if (p.act_bits == 16 && act_bytes < (size_t)kWarps * 16 * sizeof(float)) act_bytes = (size_t)kWarps * 16 * sizeof(float);
  }
  // CTAs per problem: one each, then one more at a time to the problem whose most loaded CTA has the most
  // work (a CTA owns whole runs), until every SM has one.  Work = items + the CTA's fixed cost of staging the
  // tokens' levels, in items (measured: about 1 item per token and 1024 columns from stored levels, 3 when the
  // kernel quantises x itself), so that CTAs of long-row problems get fewer items and all finish together
  const int n_sm = sm_count();
  int grid = 0;
  {
    int given[LCD_MAX_BATCH];
    long long runs[LCD_MAX_BATCH];
    int used = 0;
    for (int i = 0; i < count; ++i) {
      runs[i] = (long long)batch.p[i].n_panels * batch.p[i].n_rp;
      given[i] = 1;
      ++used;
    }
    while (used < n_sm) {
      int best = -1;
      long long best_load = 0;
      for (int i = 0; i < count; ++i) {
        const GemvProblem& gp = batch.p[i];
        const long long tokens = gp.M < 8 * MG ? gp.M : 8 * MG;
        const long long stage = (gp.act_bits == 16 ? 3 : 1) * tokens * ((long long)gp.n_kt * 256 / 1024);
        const long long load = ((runs[i] + given[i] - 1) / given[i]) * gp.pw + stage;
        if (given[i] < runs[i] && (best < 0 || load > best_load)) { best = i; best_load = load; }
      }
      if (best < 0) break;
      ++given[best];
      ++used;
    }
    for (int i = 0; i < count; ++i) {
      batch.p[i].cta0 = grid;
      batch.p[i].n_cta = given[i];
      grid += given[i];
    }
  }
  for (int i = count; i < LCD_MAX_BATCH; ++i) batch.p[i] = batch.p[0];
  for (int i = 0; i < LCD_MAX_BATCH; ++i) batch.first_cta[i] = i < count ? batch.p[i].cta0 : 0x7fffffff;
  const size_t smem = kBarBytes + combine_bytes + ring_bytes + act_bytes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (bits == 2) {
    if (kind == kFixed16) return MG == 1 ? launch_t<2, kFixed16, 1>(batch, grid, smem, status_word, s)
                                         : launch_t<2, kFixed16, 2>(batch, grid, smem, status_word, s);
    return MG == 1 ? launch_t<2, kBuckets, 1>(batch, grid, smem, status_word, s)
                   : launch_t<2, kBuckets, 2>(batch, grid, smem, status_word, s);
  }
  if (bits == 4) {      // 16-entry tables; the one-hot bucket tables would need sixteen planes
    if (kind != kFixed16) return LCD_ERR_UNSUPPORTED;
    return MG == 1 ? launch_t<4, kFixed16, 1>(batch, grid, smem, status_word, s)
                   : launch_t<4, kFixed16, 2>(batch, grid, smem, status_word, s);
  }
  if (kind == kFixed16) return MG == 1 ? launch_t<3, kFixed16, 1>(batch, grid, smem, status_word, s)
                                       : launch_t<3, kFixed16, 2>(batch, grid, smem, status_word, s);
  return MG == 1 ? launch_t<3, kBuckets, 1>(batch, grid, smem, status_word, s)
                 : launch_t<3, kBuckets, 2>(batch, grid, smem, status_word, s);
}

}  // namespace lcd
