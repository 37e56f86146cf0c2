// Shared declarations of the library's translation units (host side).
#ifndef LCD_COMMON_H_
#define LCD_COMMON_H_

#include <cstddef>
#include <cstdint>

#include "lcd.h"

namespace lcd {

constexpr uint32_t kMagic = 0x5744434Cu;  // "LCDW"
constexpr uint32_t kVersion = 1;
constexpr uint32_t kLayoutPair16x256 = 2;
constexpr uint64_t kIndexOffset = 256;
constexpr int kTileRows = 8;    // rows of one tile
constexpr int kPairRows = 16;   // two adjacent tiles form one 16-row item
constexpr int kTileK = 256;
constexpr int kKBlock = 128;
constexpr bool kHaveDenseTc = true;   // a kernel that is not built yet is skipped by LCD_ALGO_AUTO

#pragma pack(push, 1)
struct Header {
  uint32_t magic, version;
  uint64_t N, K, K_pad;
  uint32_t bits, C, layout, checksum;
  uint64_t index_offset, codebook_offset;
};
#pragma pack(pop)
static_assert(sizeof(Header) == LCD_HEADER_BYTES, "header is 64 bytes");

inline uint64_t round_up_u64(uint64_t v, uint64_t m) { return (v + m - 1) / m * m; }

bool parse_header(const void* header_host, Header* h);
size_t blob_bytes(uint64_t N, uint64_t K, int bits);

// A resolved view of a problem handed to the kernel launchers.
struct Problem {
  const uint8_t* tiles;     // device: index area
  const uint16_t* codebook; // device: [N_pad][2^bits] fp16 bits
  int64_t N, K, K_pad, N_pad;
  int bits, C;
  const uint8_t* act_idx;   // device [M][K_pad/2] (4-bit levels + 8) or [M][K_pad] signed bytes (act_bits == 8)
  int act_bits = 4;         // 4 or 8; 16 = not quantised yet: the lookup kernel does Section 4.1 itself from x
  bool dense_levels = false;          // act_idx already holds the signed bytes the int8 tensor-core kernel reads
  const void* x_fp16 = nullptr;       // act_bits == 16: device fp16 [M][ldx]
  int64_t ldx = 0;
  const float* inv_smooth = nullptr;  // act_bits == 16: device fp32 [K] or null
  const float* act_scale;   // device [M]
  int64_t M;
  float* y;
  int64_t ldy;
};

void set_cuda_error(int err);  // records cudaGetErrorString for lcd_last_cuda_error

// kernel launchers (each returns LCD_OK or LCD_ERR_CUDA / LCD_ERR_UNSUPPORTED)
lcd_status launch_smooth_quantize(const void* x, int64_t M, int64_t K, int64_t ldx, const float* inv_smooth,
                                  const float* static_scale, uint8_t* act_idx, float* act_scale, void* stream);
lcd_status launch_smooth_quantize8(const void* x, int64_t M, int64_t K, int64_t ldx, const float* inv_smooth,
                                   const float* static_scale, int8_t* act_q, float* act_scale, void* stream);
lcd_status launch_smooth_quantize8_batch(const lcd_act_problem* probs, int count, void* stream);
size_t smoothing_search_workspace_bytes(int64_t T, int64_t K, int G);
lcd_status launch_smoothing_search(const void* x, int64_t T, int64_t K, int64_t ldx, const float* wmax, const float* alphas_host,
                                   int G, void* workspace, double* mse, int32_t* best, float* inv_smooth, void* stream);
lcd_status launch_reclassify(const uint8_t* idx, const uint16_t* codebook, const float* delta_w, int64_t N, int64_t K,
                             int64_t ldw, int C, uint8_t* new_idx, double* delta_c, int32_t* counts, void* stream);
size_t dbci_workspace_bytes(int64_t n, int max_centroids);
lcd_status launch_dbci(const float* weights, int64_t n, void* workspace, float* centroids, int max_centroids,
                       int32_t* labels, float* sorted_out, lcd_dbci_result* result, void* stream);
lcd_status launch_reference(const Problem& p, void* stream);
lcd_status launch_smooth_quantize_batch(const lcd_act_problem* probs, int count, void* stream);
// The same transformation with the levels written as signed bytes [M][K_pad] in the order the int8 tensor-core kernel
// reads them for this index width (act_idx of the problems points to that buffer)
lcd_status launch_smooth_quantize_dense_levels(const lcd_act_problem* probs, int count, int bits, void* stream);
// LCD_ALGO_REGISTER_LUT / LCD_ALGO_BUCKET_LUT for up to LCD_MAX_BATCH problems of equal index width in one launch
size_t lut_gemv_workspace_bytes(const Problem* probs, int count, lcd_algo algo);
lcd_status launch_lut_gemv(const Problem* probs, int count, lcd_algo algo, void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream);
// LCD_ALGO_SHARED_BUCKET: one token, 2-bit indices, bucket tables in shared memory (4-bit levels or fp16 x)
bool lut_smem_supported(const Problem* probs, int count);
size_t lut_smem_workspace_bytes(const Problem* probs, int count);
lcd_status launch_lut_smem(const Problem* probs, int count, void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream);
// The family LCD_ALGO_AUTO stands for when every problem has at most 16 tokens.
lcd_algo resolve_small_m(const Problem* probs, int count, lcd_algo algo);
// LCD_ALGO_TC_LUT: the same arithmetic for up to 16 tokens with the looked-up bytes fed to tcgen05.mma kind::i8
size_t lut_gemv_tc_workspace_bytes(const Problem* probs, int count);
lcd_status launch_lut_gemv_tc(const Problem* probs, int count, void* workspace, size_t workspace_bytes,
                              int32_t* status_word, void* stream);
size_t dense_tc_workspace_bytes(int64_t M, int64_t K_pad);
lcd_status launch_dense_tc(const Problem& p, bool fp16_operands, void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream);

}  // namespace lcd
#endif
