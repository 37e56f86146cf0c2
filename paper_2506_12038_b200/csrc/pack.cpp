// Offline index packing (host, bit-exact).  Section 4.2, last paragraph of the LCD paper: with fewer than
// 16 centroids the clustered weights are kept as low-bit centroid indices; everything the lookup needs
// is prepared ahead of time (Section 4.1).  The byte layout is documented in include/lcd.h.
#include <cstring>
#include <vector>

#include "common.h"

namespace lcd {

static inline uint32_t payload_checksum(const uint8_t* p, size_t n) {
  uint32_t s = 0;
  for (size_t i = 0; i < n; ++i) s += p[i];
  return s;
}

bool parse_header(const void* header_host, Header* h) {
  std::memcpy(h, header_host, sizeof(Header));
  if (h->magic != kMagic || h->version != kVersion || h->layout != kLayoutPair16x256) return false;
  if (h->bits != 2 && h->bits != 3 && h->bits != 4) return false;
  if (h->C < 1 || h->C > (1u << h->bits)) return false;
  if (h->N < 1 || h->K < 1) return false;
  if (h->K_pad != round_up_u64(h->K, kTileK)) return false;
  if (h->index_offset != kIndexOffset) return false;
  const uint64_t n_pad = round_up_u64(h->N, kPairRows);
  if (h->codebook_offset != round_up_u64(kIndexOffset + n_pad * h->K_pad * h->bits / 8, 256)) return false;
  return true;
}

size_t blob_bytes(uint64_t N, uint64_t K, int bits) {
  const uint64_t n_pad = round_up_u64(N, kPairRows), k_pad = round_up_u64(K, kTileK);
  const uint64_t cb_off = round_up_u64(kIndexOffset + n_pad * k_pad * bits / 8, 256);
  return cb_off + round_up_u64(n_pad * (2ull << bits), 256);
}

// Byte offset (inside the index area) of tile (rg, kt): the tiles of rows 16rp..16rp+7 and 16rp+8..16rp+15
// are adjacent and form one 16-row item.
static inline uint64_t tile_offset(uint64_t rg, uint64_t kt, uint64_t n_kt, size_t tile_bytes) {
  return ((rg >> 1) * n_kt + kt) * 2 * tile_bytes + (rg & 1) * tile_bytes;
}

// Position of column kk (0..255) of tile row g inside a 2-bit tile: byte offset and bit shift.
static inline void locate2(int g, int kk, int* byte, int* shift) {
  const int h = kk >> 7, r = kk & 127, G = r >> 2, t = G >> 3, p = G & 7;
  *byte = 16 * (4 * g + t) + 8 * h + p;
  *shift = 2 * (r & 3);
}

// Position of column kk (0..255) of tile row g inside a 4-bit tile (two 512-byte planes, one per k-block).
static inline void locate4(int g, int kk, int* byte, int* shift) {
  const int h = kk >> 7, r = kk & 127, t = r >> 5, m = r & 31;
  *byte = 512 * h + 16 * (4 * g + t) + (m >> 1);
  *shift = 4 * (m & 1);
}

// 3-bit: the (up to three) places the bits of column kk of tile row g go to.
static inline void locate3(int g, int kk, int byte[3], int shift[3], int* contiguous) {
  const int h = kk >> 7, r = kk & 127, t = r >> 5, m = r & 31, lane = 4 * g + t;
  if (m < 24) {
    const int i = m >> 3, j = m & 7;
    byte[0] = 256 * i + 8 * lane + 4 * h + (j >> 1);
    shift[0] = 4 * (j & 1);
    *contiguous = 1;
  } else {
    const int j = m - 24;
    for (int b = 0; b < 3; ++b) {
      byte[b] = 256 * b + 8 * lane + 4 * h + (j >> 1);
      shift[b] = 4 * (j & 1) + 3;
    }
    *contiguous = 0;
  }
}

}  // namespace lcd

using namespace lcd;

extern "C" lcd_status lcd_packed_weights_bytes(int64_t N, int64_t K, int bits, size_t* bytes) {
  if (!bytes || N < 1 || K < 1) return LCD_ERR_INVALID_ARG;
  if (bits != 2 && bits != 3 && bits != 4) return LCD_ERR_UNSUPPORTED;
  *bytes = blob_bytes((uint64_t)N, (uint64_t)K, bits);
  return LCD_OK;
}

extern "C" lcd_status lcd_pack_weights(const uint8_t* idx, const uint16_t* codebook_fp16, int64_t N, int64_t K,
                                       int bits, int C, void* out, size_t out_bytes, int64_t* bad_n,
                                       int64_t* bad_k) {
  if (!idx || !codebook_fp16 || !out || N < 1 || K < 1) return LCD_ERR_INVALID_ARG;
  if (bits != 2 && bits != 3 && bits != 4) return LCD_ERR_UNSUPPORTED;
  if (C < 1 || C > (1 << bits)) return LCD_ERR_INVALID_ARG;
  const size_t total = blob_bytes((uint64_t)N, (uint64_t)K, bits);
  if (out_bytes < total) return LCD_ERR_BUFFER_TOO_SMALL;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k)
      if (idx[n * K + k] >= C) {
        if (bad_n) *bad_n = n;
        if (bad_k) *bad_k = k;
        return LCD_ERR_INDEX_RANGE;
      }
  uint8_t* blob = static_cast<uint8_t*>(out);
  std::memset(blob, 0, total);
  const uint64_t n_pad = round_up_u64(N, kPairRows), k_pad = round_up_u64(K, kTileK);
  const uint64_t n_kt = k_pad / kTileK;
  const size_t tile_bytes = kTileRows * kTileK * bits / 8;
  for (uint64_t rg = 0; rg < n_pad / kTileRows; ++rg) {
    for (uint64_t kt = 0; kt < n_kt; ++kt) {
      uint8_t* tile = blob + kIndexOffset + tile_offset(rg, kt, n_kt, tile_bytes);
      for (int g = 0; g < kTileRows; ++g) {
        const uint64_t n = rg * kTileRows + g;
        if (n >= (uint64_t)N) break;
        const uint8_t* row = idx + n * K;
        for (int kk = 0; kk < kTileK; ++kk) {
          const uint64_t k = kt * kTileK + kk;
          if (k >= (uint64_t)K) break;
          const uint32_t v = row[k];
          if (bits == 2) {
            int byte, shift;
            locate2(g, kk, &byte, &shift);
            tile[byte] |= (uint8_t)(v << shift);
          } else if (bits == 4) {
            int byte, shift;
            locate4(g, kk, &byte, &shift);
            tile[byte] |= (uint8_t)(v << shift);
          } else {
            int byte[3], shift[3], contiguous;
            locate3(g, kk, byte, shift, &contiguous);
            if (contiguous) {
              tile[byte[0]] |= (uint8_t)(v << shift[0]);
            } else {
              for (int b = 0; b < 3; ++b) tile[byte[b]] |= (uint8_t)(((v >> b) & 1u) << shift[b]);
            }
          }
        }
      }
    }
  }
  const uint64_t cb_off = round_up_u64(kIndexOffset + n_pad * k_pad * bits / 8, 256);
  const int cs = 1 << bits;
  uint16_t* cb = reinterpret_cast<uint16_t*>(blob + cb_off);
  for (int64_t n = 0; n < N; ++n)
    for (int w = 0; w < C; ++w) cb[n * cs + w] = codebook_fp16[n * C + w];
  Header h;
  std::memset(&h, 0, sizeof(h));
  h.magic = kMagic;
  h.version = kVersion;
  h.N = (uint64_t)N;
  h.K = (uint64_t)K;
  h.K_pad = k_pad;
  h.bits = (uint32_t)bits;
  h.C = (uint32_t)C;
  h.layout = kLayoutPair16x256;
  h.index_offset = kIndexOffset;
  h.codebook_offset = cb_off;
  h.checksum = payload_checksum(blob + sizeof(Header), total - sizeof(Header));
  std::memcpy(blob, &h, sizeof(h));
  return LCD_OK;
}

extern "C" lcd_status lcd_unpack_weights(const void* blob_v, size_t blob_bytes_in, uint8_t* idx,
                                         uint16_t* codebook_fp16, int64_t* N, int64_t* K, int* bits, int* C) {
  if (!blob_v) return LCD_ERR_INVALID_ARG;
  if (blob_bytes_in < sizeof(Header)) return LCD_ERR_BAD_BLOB;
  const uint8_t* blob = static_cast<const uint8_t*>(blob_v);
  Header h;
  if (!parse_header(blob, &h)) return LCD_ERR_BAD_BLOB;
  const size_t total = blob_bytes(h.N, h.K, (int)h.bits);
  if (blob_bytes_in < total) return LCD_ERR_BAD_BLOB;
  if (payload_checksum(blob + sizeof(Header), total - sizeof(Header)) != h.checksum) return LCD_ERR_BAD_BLOB;
  if (N) *N = (int64_t)h.N;
  if (K) *K = (int64_t)h.K;
  if (bits) *bits = (int)h.bits;
  if (C) *C = (int)h.C;
  const uint64_t n_kt = h.K_pad / kTileK;
  const size_t tile_bytes = kTileRows * kTileK * h.bits / 8;
  if (idx) {
    for (uint64_t n = 0; n < h.N; ++n) {
      const uint64_t rg = n / kTileRows;
      const int g = (int)(n % kTileRows);
      for (uint64_t k = 0; k < h.K; ++k) {
        const uint8_t* tile = blob + h.index_offset + tile_offset(rg, k / kTileK, n_kt, tile_bytes);
        const int kk = (int)(k % kTileK);
        uint32_t v;
        if (h.bits == 2) {
          int byte, shift;
          locate2(g, kk, &byte, &shift);
          v = (tile[byte] >> shift) & 3u;
        } else if (h.bits == 4) {
          int byte, shift;
          locate4(g, kk, &byte, &shift);
          v = (tile[byte] >> shift) & 15u;
        } else {
          int byte[3], shift[3], contiguous;
          locate3(g, kk, byte, shift, &contiguous);
          if (contiguous) {
            v = (tile[byte[0]] >> shift[0]) & 7u;
          } else {
            v = 0;
            for (int b = 0; b < 3; ++b) v |= ((tile[byte[b]] >> shift[b]) & 1u) << b;
          }
        }
        idx[n * h.K + k] = (uint8_t)v;
      }
    }
  }
  if (codebook_fp16) {
    const uint16_t* cb = reinterpret_cast<const uint16_t*>(blob + h.codebook_offset);
    const int cs = 1 << h.bits;
    for (uint64_t n = 0; n < h.N; ++n)
      for (uint32_t w = 0; w < h.C; ++w) codebook_fp16[n * h.C + w] = cb[n * cs + w];
  }
  return LCD_OK;
}
