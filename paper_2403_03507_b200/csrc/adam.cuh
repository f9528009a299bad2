// Adam-on-R kernels and the 8-bit block-wise state format: declarations.
#pragma once

#include "common.cuh"
#include "q8_code.cuh"

namespace galore {

constexpr int kStateTileCols = 64;    // a quantisation block is a tile of q_block / 64 rows x 64 columns of the state

// One layer's share of a grouped Adam launch.  The state (shape of R: rows x cols) is walked in tiles
// of tile_rows x 64; R partials, N and the state arrays are row-major with their own row pitches.
struct AdamItem {
  const float* Rpart;      // split-K partials of R
  int splits;
  int64_t split_stride;
  int rows, cols;          // shape of R, M, V
  int64_t r_ld, n_ld, s_ld;  // row pitches (elements) of Rpart, Nout and the state arrays
  float *M, *V;            // fp32 moments, or
  uint8_t *Mc, *Vc;        // 8-bit codes with
  float *Mam, *Vam;        // one absmax per tile, tile (I, J) at I * tiles_c + J
  void* Nout;              // normalised update (fp32 or bf16)
  int tiles_c;             // set by adam_group_add: ceil(cols / 64)
  int vec;                 // set by adam_group_add: bases and pitches allow the vector accesses of an interior tile
  int sub_r0, sub_c0, sub_nc;  // the item covers the tiles (sub_r0 + b / sub_nc, sub_c0 + b % sub_nc), b = 0, 1, ...
  uint32_t sub_magic;      // ceil(2^32 / sub_nc) when b / sub_nc = mulhi(b, sub_magic) for every b of the item, else 0
  AdamParams p;
  int32_t* status;
};
constexpr int kAdamGroup = 32;
struct AdamGroup {
  AdamItem item[kAdamGroup];
  int block_end[kAdamGroup];   // running total of tiles
  int count;
};
// all items of a group share the state format, the quantisation block and the dtype of N
galore_status_t adam_group_add(AdamGroup& g, const AdamItem& item, int32_t state_fmt, int q_block);
galore_status_t launch_adam_group(const AdamGroup& g, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st);
// one layer
galore_status_t launch_adam(const AdamItem& item, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st);

// Pitches and sizes of a layer's state arrays.  fp32 moments: rows of ceil8(cols) floats; 8-bit codes:
// rows of ceil32(cols) bytes, plus ceil(rows / (q_block / 64)) * ceil(cols / 64) absmax values.
inline int64_t state_pitch(int32_t state_fmt, int64_t cols) {
  return state_fmt == GALORE_STATE_Q8_BLOCK ? (cols + 31) / 32 * 32 : (cols + 7) / 8 * 8;
}
inline int64_t state_tiles(int64_t rows, int64_t cols, int q_block) {
  return ceil_div(rows, q_block / kStateTileCols) * ceil_div(cols, kStateTileCols);
}

// x (rows x cols fp32, pitch ldx) -> codes (pitch ldc) and one absmax per tile_rows x tile_cols tile
galore_status_t launch_q8_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, int is_signed, int tile_rows,
                                   int tile_cols, uint8_t* codes, int64_t ldc, float* absmax, cudaStream_t st);
galore_status_t launch_q8_dequantize(const uint8_t* codes, int64_t ldc, const float* absmax, int64_t rows, int64_t cols,
                                     int is_signed, int tile_rows, int tile_cols, float* out, int64_t ldo, cudaStream_t st);
galore_status_t q8_ensure_tables();
galore_status_t q8_table_ptrs(Q8TablePtrs* out);   // device addresses on the current device (fills the tables first)
void q8_host_codebook(bool is_signed, float* out256);

}  // namespace galore
