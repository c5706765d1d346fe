// Structures shared by the host planner and the kernels of the Muon step.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace muon {

// Tile shape of the Newton-Schulz GEMM kernel.
constexpr int kBM = 128;     // output tile rows  (UMMA M)
constexpr int kBN = 128;     // output tile cols  (UMMA N)
constexpr int kBK = 64;      // K elements per pipeline stage (128 bytes of bf16)
constexpr int kStages = 5;   // TMA -> UMMA pipeline depth
constexpr int kGemmThreads = 192;  // warp 0: TMA, warp 1: UMMA, warps 2-5: epilogue

// Tile of the streaming momentum kernel (source orientation rows x cols).
constexpr int kSTR = 64;
constexpr int kSTC = 128;
constexpr int kStreamThreads = 512;

// Per-matrix descriptor in device memory.
struct MatDesc {
  void* w;
  const void* g;
  float* m;
  long long ld_w, ld_g, ld_m;
  int rows, cols;
  int transposed;  // rows > cols: Newton-Schulz runs on the transpose
  int vec_ok;      // all three of W, G, M allow 16-byte vector access
  int global_index;  // position in the caller's group list (groups in order)
  int pad_;
};

// Per-matrix scalars written by the norm finalisation kernel.
struct MatScal {
  float inv_norm;     // s = 1 / (||U||_F + eps)
  float inv_norm_sq;  // s^2
  float norm;         // ||U||_F
  int nonfinite;      // 1 if the norm is NaN/Inf
};

// Device status word: {code, first matrix index}.
struct DevStatus {
  int code;
  int matrix;
};

enum GemmMode { kGram = 0, kPoly = 1, kComb = 2 };

struct GemmParams {
  CUtensorMap map_a;      // operand A rows (K-major), box {64, 128}, 128B swizzle
  CUtensorMap map_b;      // operand B: K-major box {64, 128}, or MN-major box {64, 64}
  CUtensorMap map_in;     // epilogue input tile, box {64, 128}, 128B swizzle
  CUtensorMap map_out;    // output tile, box {64, 128}, 128B swizzle
  CUtensorMap map_out_t;  // transposed output tile, box {128, 128}, no swizzle
  int mode;
  int out_rows, out_cols;  // output extent per matrix (m x m, or m x n)
  int k;                   // contraction length
  int count;               // matrices in this launch
  int nb_i, nb_j;          // 128-tiles along rows / cols of the output
  int tiles_per_matrix;
  int symmetric;      // upper-triangle tiles only, mirrored
  int has_in;         // epilogue reads an input tile
  int write_direct;   // store the bf16 tile through map_out
  int write_t;        // store the transposed bf16 tile through map_out_t (off-diagonal only
                      // when symmetric)
  int scale_kind;     // 0: none, 1: multiply by s^2 of the matrix, 2: multiply by s
  int last;           // fused weight update in the epilogue
  int b_mn_major;     // operand B is MN-major (read from X itself)
  float c_acc, c_in;  // tile = scale * (c_acc * acc + c_in * in)
  // fused update (last iteration)
  float upd_scale;  // -lr * rms_scale * sqrt(max(rows, cols))
  float decay;      // 1 - lr * wd
  int w_fp32;
  const MatDesc* descs;  // chunk-relative
  const MatScal* scal;   // chunk-relative
  DevStatus* status;
};

// One entry of a tile table of the CTA-pair kernel: the pair covers row blocks
// 2*p and 2*p+1 (128 rows each, one per CTA) and `nbw` (1 or 2) column blocks
// starting at block `jb`.
struct PairTile {
  short p, jb, nbw, pad_;
};

// Parameters of the CTA-pair Newton-Schulz GEMM kernel (cta_group::2).
struct PairGemmParams {
  CUtensorMap map_a;      // operand A rows, box {64 K, 128 rows}, 128B swizzle
  CUtensorMap map_b;      // operand B, box {64, 64}, 128B swizzle (K-major: {K, rows};
                          // MN-major: {N, K})
  CUtensorMap map_in;     // epilogue input, box {64, 128}, 128B swizzle
  CUtensorMap map_out;    // output, box {64, 128}, 128B swizzle
  CUtensorMap map_out_t;  // mirrored output, box {128, 64}, no swizzle
  const PairTile* tiles;  // tile table of one matrix
  int tiles_per_matrix;
  int count;       // matrices in this launch
  int k;           // contraction length
  int symmetric;   // upper-triangle blocks only, mirrored
  int has_in;
  int write_direct;
  int scale_kind;  // 0: none, 1: s^2, 2: s
  int last;        // fused weight update
  int b_mn_major;
  float c_acc, c_in;
  float upd_scale, decay;
  int w_fp32;
  const MatDesc* descs;
  const MatScal* scal;
  DevStatus* status;
  unsigned* debug;  // optional: TMEM base addresses seen by each CTA (test builds)
};

struct StreamParams {
  const MatDesc* descs;
  float* partials;  // [count][tiles_per_matrix]
  __nv_bfloat16* x;   // [count][m][ldx], short side first
  __nv_bfloat16* xt;  // [count][n][ldxt] or nullptr
  long long x_stride, xt_stride;  // elements per matrix
  int ldx, ldxt;
  int count;
  int tiles_per_matrix;
  float mu;
  int nesterov;
};

}  // namespace muon
