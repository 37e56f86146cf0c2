// Reference-grade lookup-and-accumulate kernel (Section 4.2 of the LCD paper, plain form): for every weight,
// read its centroid index from the tiled blob, look the centroid up in the row codebook, multiply by the
// token's activation level and accumulate in fp32.  Works for every M, N, K and every index width; it is the
// library's correctness anchor, not a fast path.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "common.h"
#include "layout.cuh"

namespace lcd {

// CTA = 8 warps = the 8 rows of one row group; lane = token inside a block of 32 tokens.
__global__ void __launch_bounds__(256)
reference_kernel(const uint8_t* __restrict__ tiles, const uint16_t* __restrict__ codebook, int64_t N, int64_t K,
                 int64_t K_pad, int bits, int act_bits, const uint8_t* __restrict__ act_idx,
                 const float* __restrict__ act_scale,
                 int64_t M, float* __restrict__ y, int64_t ldy) {
  __shared__ float s_cb[8][16];
  const int g = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t rg = blockIdx.x;
  const int64_t n = rg * 8 + g;
  const int64_t m = (int64_t)blockIdx.y * 32 + lane;
  const int cs = 1 << bits;
  if (lane < cs) s_cb[g][lane] = __half2float(__ushort_as_half(codebook[n * cs + lane]));
  __syncwarp();
  const int64_t n_kt = K_pad / kTileK;
  const size_t tile_bytes = (size_t)kTileRows * kTileK * bits / 8;
  const uint8_t* act_row = act_idx + (m < M ? m : 0) * (act_bits == 8 ? K_pad : K_pad / 2);
  float acc = 0.0f;
  for (int64_t k = 0; k < K; ++k) {
    const uint8_t* tile = tiles + (((rg >> 1) * n_kt + k / kTileK) * 2 + (rg & 1)) * tile_bytes;
    const int kk = (int)(k % kTileK);
    const uint32_t w = bits == 2 ? tile_index_2bit(tile, g, kk) : bits == 3 ? tile_index_3bit(tile, g, kk) : tile_index_4bit(tile, g, kk);
    int q;
    if (act_bits == 8) {
      q = (int)(int8_t)act_row[k];
    } else {
      const uint32_t byte = act_row[k >> 1];
      q = (int)((byte >> (4 * (k & 1))) & 15u) - 8;
    }
    acc = fmaf((float)q, s_cb[g][w], acc);
  }
  if (m < M && n < N) y[m * ldy + n] = act_scale[m] * acc;
}

lcd_status launch_reference(const Problem& p, void* stream) {
  dim3 grid((unsigned)(p.N_pad / kTileRows), (unsigned)((p.M + 31) / 32));
  reference_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      p.tiles, p.codebook, p.N, p.K, p.K_pad, p.bits, p.act_bits, p.act_idx, p.act_scale, p.M, p.y, p.ldy);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_cuda_error((int)e);
    return LCD_ERR_CUDA;
  }
  return LCD_OK;
}

}  // namespace lcd
