// LUT-GEMV for M <= 16 with the row codebook held as a byte table in registers (Section 4.2 of the LCD paper:
// values are fetched from a small table by weight index and accumulated; no weight is ever multiplied in
// floating point).  Per output row the fp16 centroids are turned into 16-bit fixed point, split into a high
// (signed) and a low (unsigned) byte table; one PRMT looks up four weights at once (the weight index nibbles
// are the selector), and the looked-up bytes are accumulated against the token's activation levels with
// integer dot products (DP4A).  Bucket structure: everything a row needs is its own 2^bits-entry table, so all
// rows proceed in parallel.  y = s_q * 2^e_n * (256 * accH + accL).
//
// Thread mapping follows the tile layout: a warp owns one row group (8 rows), lane 4g+t owns quarter t
// (32 of every 128 columns) of row g.  A CTA of 8 warps covers RGC row groups x KS interleaved column slices;
// slice partial sums (exact integers) are combined through shared memory in a fixed order.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"

namespace lcd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSmem = 200 * 1024;

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Activation levels of one token chunk as signed bytes in shared memory, ordered the way the lookups emit
// weights.  Source: packed 4-bit a = q + 8, column k even in the low nibble.  One 32-bit source word = 8 columns.
//   2 bit: per 32-column quarter the 8 output words are [E(w0) E(w1) O(w0) O(w1) E(w2) E(w3) O(w2) O(w3)],
//          E(w)/O(w) = the even/odd columns of source word w.
//   3 bit: natural column order.
template <int BITS>
__device__ __forceinline__ void stage_activations(uint32_t* q_s, const uint8_t* act_row, int64_t k0, int n_cols,
                                                  bool valid, int tid) {
  const uint32_t* src = reinterpret_cast<const uint32_t*>(act_row + (k0 >> 1));
  for (int j = tid; j < n_cols / 8; j += kThreads) {
    const uint32_t a = valid ? src[j] : 0x88888888u;
    uint32_t e = a & 0x0f0f0f0fu, o = (a >> 4) & 0x0f0f0f0fu;
    e = (e + 0x78787878u) ^ 0x80808080u;   // per byte a - 8 without cross-byte borrow
    o = (o + 0x78787878u) ^ 0x80808080u;
    const int quarter = j >> 2, w = j & 3;
    if (BITS == 2) {
      q_s[quarter * 8 + (w & 1) + 4 * (w >> 1)] = e;
      q_s[quarter * 8 + 2 + (w & 1) + 4 * (w >> 1)] = o;
    } else {
      q_s[quarter * 8 + 2 * w] = prmt(e, o, 0x5140u);
      q_s[quarter * 8 + 2 * w + 1] = prmt(e, o, 0x7362u);
    }
  }
}

template <int BITS>
struct Tables {
  uint32_t h[BITS == 2 ? 1 : 2], l[BITS == 2 ? 1 : 2];
  float scale;
};

// 16-bit fixed-point byte tables of one row's codebook: value = (256*H + L) * scale, H signed, L unsigned.
template <int BITS>
__device__ __forceinline__ Tables<BITS> build_tables(const uint16_t* cb_row) {
  constexpr int C = 1 << BITS;
  float v[C];
  if (BITS == 2) {
    const uint2 raw = *reinterpret_cast<const uint2*>(cb_row);
    const __half2* h = reinterpret_cast<const __half2*>(&raw);
    const float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
  } else {
    const uint4 raw = *reinterpret_cast<const uint4*>(cb_row);
    const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 a = __half22float2(h[i]);
      v[2 * i] = a.x; v[2 * i + 1] = a.y;
    }
  }
  float mx = 0.0f;
#pragma unroll
  for (int i = 0; i < C; ++i) mx = fmaxf(mx, fabsf(v[i]));
  int ex = 0;
  (void)frexpf(mx, &ex);                       // mx < 2^ex
  const float up = scalbnf(1.0f, 15 - ex);     // mx * up < 32768
  Tables<BITS> T;
  T.scale = scalbnf(1.0f, ex - 15);
  uint32_t hb[2] = {0, 0}, lb[2] = {0, 0};
#pragma unroll
  for (int i = 0; i < C; ++i) {
    const int f = __float2int_rn(v[i] * up);
    hb[i >> 2] |= ((uint32_t)(f >> 8) & 0xffu) << (8 * (i & 3));
    lb[i >> 2] |= ((uint32_t)f & 0xffu) << (8 * (i & 3));
  }
  T.h[0] = hb[0]; T.l[0] = lb[0];
  if (BITS == 3) { T.h[1] = hb[1]; T.l[1] = lb[1]; }
  return T;
}

template <int BITS, int MT>
__device__ __forceinline__ void lookup4(const Tables<BITS>& T, uint32_t sel, const uint32_t (&q)[MT], int (&accH)[MT],
                                        int (&accL)[MT]) {
  uint32_t hv, lv;
  if (BITS == 2) {
    hv = prmt(T.h[0], T.l[0], sel);
    lv = prmt(T.l[0], T.h[0], sel);
  } else {
    hv = prmt(T.h[0], T.h[1], sel);
    lv = prmt(T.l[0], T.l[1], sel);
  }
#pragma unroll
  for (int m = 0; m < MT; ++m) {
    accH[m] = dp4a_ss(hv, q[m], accH[m]);
    accL[m] = dp4a_us(lv, q[m], accL[m]);
  }
}

// One k-block (128 columns) of one row group: lane (g,t) consumes its 32 weights.
// r[]: 2 bit: the lane's 8 bytes (2 words); 3 bit: the 3 record words.
template <int BITS, int MT>
__device__ __forceinline__ void kblock(const Tables<BITS>& T, const uint32_t* r, const uint32_t* q_quarter,
                                       int chunk_words, uint32_t selU0, uint32_t selU1, int (&accH)[MT],
                                       int (&accL)[MT]) {
  uint4 qa[MT], qb[MT];
#pragma unroll
  for (int m = 0; m < MT; ++m) {
    qa[m] = *reinterpret_cast<const uint4*>(q_quarter + (size_t)m * chunk_words);
    qb[m] = *reinterpret_cast<const uint4*>(q_quarter + (size_t)m * chunk_words + 4);
  }
  uint32_t q[MT];
  if (BITS == 2) {
    const uint32_t u0 = prmt(r[0], r[1], selU0), u1 = prmt(r[0], r[1], selU1);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const uint32_t u = half ? u1 : u0;
      const uint32_t s0 = u & 0x33333333u, s1 = (u >> 2) & 0x33333333u;
#pragma unroll
      for (int m = 0; m < MT; ++m) q[m] = half ? qb[m].x : qa[m].x;
      lookup4<BITS, MT>(T, s0, q, accH, accL);
#pragma unroll
      for (int m = 0; m < MT; ++m) q[m] = half ? qb[m].y : qa[m].y;
      lookup4<BITS, MT>(T, s0 >> 16, q, accH, accL);
#pragma unroll
      for (int m = 0; m < MT; ++m) q[m] = half ? qb[m].z : qa[m].z;
      lookup4<BITS, MT>(T, s1, q, accH, accL);
#pragma unroll
      for (int m = 0; m < MT; ++m) q[m] = half ? qb[m].w : qa[m].w;
      lookup4<BITS, MT>(T, s1 >> 16, q, accH, accL);
    }
  } else {
    const uint32_t d0 = r[0] & 0x77777777u, d1 = r[1] & 0x77777777u, d2 = r[2] & 0x77777777u;
    const uint32_t ex = ((r[0] & 0x88888888u) >> 3) | ((r[1] & 0x88888888u) >> 2) | ((r[2] & 0x88888888u) >> 1);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qa[m].x;
    lookup4<BITS, MT>(T, d0, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qa[m].y;
    lookup4<BITS, MT>(T, d0 >> 16, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qa[m].z;
    lookup4<BITS, MT>(T, d1, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qa[m].w;
    lookup4<BITS, MT>(T, d1 >> 16, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qb[m].x;
    lookup4<BITS, MT>(T, d2, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qb[m].y;
    lookup4<BITS, MT>(T, d2 >> 16, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qb[m].z;
    lookup4<BITS, MT>(T, ex, q, accH, accL);
#pragma unroll
    for (int m = 0; m < MT; ++m) q[m] = qb[m].w;
    lookup4<BITS, MT>(T, ex >> 16, q, accH, accL);
  }
}

// Persistent CTAs of 8 warps.  Work unit = (row group, column slice); a CTA iteration takes 8 consecutive units,
// i.e. 8/KS row groups x KS slices, so the slices of a row group meet in the same CTA and are combined through
// shared memory.  A warp first issues the loads of up to kBatch tiles of its slice (memory-level parallelism),
// then consumes them.
constexpr int kBatch = 8;

template <int BITS>
struct TileRegs {
  uint32_t w[BITS * 2];   // 2 bit: 4 words (16 B); 3 bit: 6 words (3 x 8 B)
};

template <int BITS>
__device__ __forceinline__ TileRegs<BITS> load_tile(const uint8_t* tile, int lane) {
  TileRegs<BITS> r;
  if (BITS == 2) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(tile + 16 * lane));
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
  } else {
    const uint2 a = __ldg(reinterpret_cast<const uint2*>(tile + 8 * lane));
    const uint2 b = __ldg(reinterpret_cast<const uint2*>(tile + 256 + 8 * lane));
    const uint2 c = __ldg(reinterpret_cast<const uint2*>(tile + 512 + 8 * lane));
    r.w[0] = a.x; r.w[1] = b.x; r.w[2] = c.x; r.w[3] = a.y; r.w[4] = b.y; r.w[5] = c.y;
  }
  return r;
}

template <int BITS, int MT>
__global__ void __launch_bounds__(kThreads, 2)
register_lut_kernel(const uint8_t* __restrict__ tiles, const uint16_t* __restrict__ codebook, int64_t N,
                    int64_t n_rg, int n_kt, const uint8_t* __restrict__ act_idx,
                    const float* __restrict__ act_scale, int M, float* __restrict__ y, int64_t ldy, int KS,
                    int chunk_tiles, int n_chunks) {
  extern __shared__ __align__(16) uint32_t smem[];
  const int chunk_words = chunk_tiles * (kTileK / 4);           // words of staged bytes per token
  uint32_t* q_s = smem;                                         // [MT][chunk_words]
  int* red_s = reinterpret_cast<int*>(smem + (size_t)MT * chunk_words);  // [8 warps][MT][8 rows][2]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int RGC = kWarps / KS;
  const int ks = warp % KS, rgi = warp / KS;
  constexpr int TILE_BYTES = kTileRows * kTileK * BITS / 8;
  const int64_t K_pad = (int64_t)n_kt * kTileK;
  uint32_t selU0 = 0, selU1 = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    selU0 |= (uint32_t)((j - g) & 7) << (4 * j);
    selU1 |= (uint32_t)((4 + j - g) & 7) << (4 * j);
  }
  const int slice_tiles = (n_kt + KS - 1) / KS;
  const int64_t n_rounds = (n_rg + RGC - 1) / RGC;
  bool staged = false;
  for (int64_t round = blockIdx.x; round < n_rounds; round += gridDim.x) {
    const int64_t rg = round * RGC + rgi;
    const bool active = rg < n_rg;
    const uint8_t* row_tiles = tiles + (size_t)(active ? rg : 0) * n_kt * TILE_BYTES;
    int accH[MT], accL[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) accH[m] = accL[m] = 0;
    Tables<BITS> T;
    bool have_tables = false;
    for (int c = 0; c < n_chunks; ++c) {
      const int kt0 = c * chunk_tiles;
      const int kt1 = min(n_kt, kt0 + chunk_tiles);
      // this warp's tiles inside the chunk
      const int my0 = max(kt0, ks * slice_tiles), my1 = min(kt1, min(n_kt, (ks + 1) * slice_tiles));
      TileRegs<BITS> buf[kBatch];
      int kt = my0;
      if (active) {
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
          if (kt + b < my1) buf[b] = load_tile<BITS>(row_tiles + (size_t)(kt + b) * TILE_BYTES, lane);
      }
      if (active && !have_tables) {
        T = build_tables<BITS>(codebook + (rg * 8 + g) * (1 << BITS));
        have_tables = true;
      }
      if (n_chunks > 1 || !staged) {
        __syncthreads();
#pragma unroll
        for (int m = 0; m < MT; ++m)
          stage_activations<BITS>(q_s + (size_t)m * chunk_words, act_idx + (size_t)(m < M ? m : 0) * (K_pad / 2),
                                  (int64_t)kt0 * kTileK, (kt1 - kt0) * kTileK, m < M, tid);
        __syncthreads();
        staged = true;
      }
      if (active) {
        while (kt < my1) {
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            if (kt + b < my1) {
              const uint32_t* q_tile = q_s + (size_t)(kt + b - kt0) * (kTileK / 4) + t * 8;
              if (BITS == 2) {
                kblock<BITS, MT>(T, &buf[b].w[0], q_tile, chunk_words, selU0, selU1, accH, accL);
                kblock<BITS, MT>(T, &buf[b].w[2], q_tile + kKBlock / 4, chunk_words, selU0, selU1, accH, accL);
              } else {
                kblock<BITS, MT>(T, &buf[b].w[0], q_tile, chunk_words, selU0, selU1, accH, accL);
                kblock<BITS, MT>(T, &buf[b].w[3], q_tile + kKBlock / 4, chunk_words, selU0, selU1, accH, accL);
              }
            }
          }
          kt += kBatch;
          if (kt < my1) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b)
              if (kt + b < my1) buf[b] = load_tile<BITS>(row_tiles + (size_t)(kt + b) * TILE_BYTES, lane);
          }
        }
      }
    }
    // combine the four quarters of a row (lanes t = 0..3), then the KS slices through shared memory
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      accH[m] += __shfl_xor_sync(0xffffffffu, accH[m], 1);
      accL[m] += __shfl_xor_sync(0xffffffffu, accL[m], 1);
      accH[m] += __shfl_xor_sync(0xffffffffu, accH[m], 2);
      accL[m] += __shfl_xor_sync(0xffffffffu, accL[m], 2);
    }
    if (KS > 1) {
      __syncthreads();   // red_s free again (previous round's readers are done)
      if (t == 0) {
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          red_s[((warp * MT + m) * 8 + g) * 2 + 0] = active ? accH[m] : 0;
          red_s[((warp * MT + m) * 8 + g) * 2 + 1] = active ? accL[m] : 0;
        }
      }
      __syncthreads();
    }
    // warps with ks == 0 finish their row group: lane (g,t) handles tokens t, t+4, ...
    if (ks == 0 && active) {
      const int64_t n = rg * 8 + g;
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        if ((m & 3) == t && m < M) {
          int h = accH[m], l = accL[m];
          if (KS > 1) {
            h = 0; l = 0;
            for (int s = 0; s < KS; ++s) {
              h += red_s[(((rgi * KS + s) * MT + m) * 8 + g) * 2 + 0];
              l += red_s[(((rgi * KS + s) * MT + m) * 8 + g) * 2 + 1];
            }
          }
          if (n < N) y[(size_t)m * ldy + n] = act_scale[m] * T.scale * ((float)h * 256.0f + (float)l);
        }
      }
    }
  }
}

template <int BITS, int MT>
lcd_status launch_t(const Problem& p, cudaStream_t stream) {
  const int n_kt = (int)(p.K_pad / kTileK);
  const int64_t n_rg = p.N_pad / kTileRows;
  // column slices per row group: minimise (waves of CTAs) x (tiles per slice + one tile of fixed cost)
  int KS = 1;
  {
    int64_t best = -1;
    for (int cand = 1; cand <= 8; cand *= 2) {
      const int slice = (n_kt + cand - 1) / cand;
      if (cand > 1 && slice < 2) break;
      const int64_t rounds = (n_rg + kWarps / cand - 1) / (kWarps / cand);
      const int64_t cost = ((rounds + 295) / 296) * (slice + 1);
      if (best < 0 || cost < best) { best = cost; KS = cand; }
    }
  }
  const size_t red_bytes = (size_t)kWarps * MT * 8 * 2 * sizeof(int);
  int chunk_tiles = n_kt;
  const size_t per_tile = (size_t)MT * kTileK;
  if (per_tile * chunk_tiles + red_bytes > (size_t)kMaxSmem) chunk_tiles = (int)((kMaxSmem - red_bytes) / per_tile);
  const int n_chunks = (n_kt + chunk_tiles - 1) / chunk_tiles;
  const size_t smem = per_tile * chunk_tiles + red_bytes;
  auto kern = register_lut_kernel<BITS, MT>;
  static bool attr_set = false;   // per template instance
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem + 1024);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
    attr_set = true;
  }
  const int RGC = kWarps / KS;
  const int64_t n_rounds = (n_rg + RGC - 1) / RGC;
  int per_sm = (int)((size_t)(220 * 1024) / (smem + 1024));
  per_sm = per_sm < 1 ? 1 : (per_sm > 2 ? 2 : per_sm);
  const int64_t grid = n_rounds < (int64_t)148 * per_sm ? n_rounds : (int64_t)148 * per_sm;
  kern<<<(unsigned)grid, kThreads, smem, stream>>>(p.tiles, p.codebook, p.N, n_rg, n_kt, p.act_idx, p.act_scale,
                                                   (int)p.M, p.y, p.ldy, KS, chunk_tiles, n_chunks);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

template <int BITS>
lcd_status launch_bits(const Problem& p, cudaStream_t stream) {
  if (p.M == 1) return launch_t<BITS, 1>(p, stream);
  if (p.M == 2) return launch_t<BITS, 2>(p, stream);
  if (p.M <= 4) return launch_t<BITS, 4>(p, stream);
  if (p.M <= 8) return launch_t<BITS, 8>(p, stream);
  return launch_t<BITS, 16>(p, stream);
}

}  // namespace

lcd_status launch_register_lut(const Problem& p, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return p.bits == 2 ? launch_bits<2>(p, s) : launch_bits<3>(p, s);
}

}  // namespace lcd
