// Device-side view of the tiled index layout (documented in include/lcd.h).
#ifndef LCD_LAYOUT_CUH_
#define LCD_LAYOUT_CUH_

#include <cstdint>

namespace lcd {

// Index of column kk (0..255) of row g (0..7) inside one 512-byte 2-bit tile.
__device__ __forceinline__ uint32_t tile_index_2bit(const uint8_t* tile, int g, int kk) {
  const int h = kk >> 7, r = kk & 127, G = r >> 2, t = G >> 3, p = G & 7;
  return (tile[16 * (4 * g + t) + 8 * h + p] >> (2 * (r & 3))) & 3u;
}

// Index of column kk (0..255) of row g (0..7) inside one 768-byte 3-bit tile.
__device__ __forceinline__ uint32_t tile_index_3bit(const uint8_t* tile, int g, int kk) {
  const int h = kk >> 7, r = kk & 127, t = r >> 5, m = r & 31, lane = 4 * g + t;
  const uint32_t* base = reinterpret_cast<const uint32_t*>(tile) + 2 * lane + h;  // word b is at +64*b
  if (m < 24) return (base[64 * (m >> 3)] >> (4 * (m & 7))) & 7u;
  const int sh = 4 * (m - 24) + 3;
  return ((base[0] >> sh) & 1u) | (((base[64] >> sh) & 1u) << 1) | (((base[128] >> sh) & 1u) << 2);
}

// Index of column kk (0..255) of row g (0..7) inside one 1024-byte 4-bit tile.
__device__ __forceinline__ uint32_t tile_index_4bit(const uint8_t* tile, int g, int kk) {
  const int h = kk >> 7, r = kk & 127, t = r >> 5, m = r & 31;
  return (tile[512 * h + 16 * (4 * g + t) + (m >> 1)] >> (4 * (m & 1))) & 15u;
}

}  // namespace lcd
#endif
