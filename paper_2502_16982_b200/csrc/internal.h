// Structures shared by the host planner and the kernels of the Muon step.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace muon {

// Newton-Schulz GEMM kernel: a CTA pair owns a 256-row x (128 or 256)-column
// output tile; operands are staged 64 K-elements (128 bytes of bf16) at a time.
constexpr int kBM = 128;     // output rows per CTA (UMMA M = 256 over the pair)
constexpr int kBK = 64;      // K elements per pipeline stage
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
  void* w_shadow;    // optional bf16 copy of fp32 weights, written with every update
  long long ld_ws;
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

// One entry of a tile table.  For rank r in {0, 1} the CTA pair computes the 128
// output rows of row block i[r] of matrix (first matrix of the unit + dm[r])
// against N = 128 * nbw output columns:
//   nbw == 2: accumulator columns [0, 128) are column block j[0], [128, 256)
//             column block j[1]; CTA r stages the operand-B rows of block j[r],
//             taken from ITS matrix;
//   nbw == 1: the columns are block j[0]; each CTA stages 64 of its rows.
// half != 0: a half-height tile (UMMA M = 128 over the pair instead of 256).  The
// pair computes ONE row block, i[0], its upper 64 rows in CTA 0 and its lower 64
// in CTA 1, against the same columns; dm[0] names the matrix.  It costs half a
// full tile's tensor-core time, so a row block that has no partner (an odd
// number of row blocks, a lone diagonal block) wastes nothing.
// keep[r] bit h set: the 128 x 128 block (rows of CTA r, column half h) is
// stored (half-height tiles: keep[0] bit h for column half h of the row block).  The other blocks of the product are computed and dropped: a block
// below the diagonal of a symmetric result, or the cross terms of a tile whose
// two CTAs work on different matrices.
// The row blocks (and, for a symmetric operand B, the column blocks) of one
// entry are equal or neighbours, because one instruction reads an operand of
// both CTAs in one layout (see TilePlan in ns_gemm.cu).
struct PairTile {
  short i[2];
  short j[2];
  unsigned char nbw;
  unsigned char dm[2];
  unsigned char keep[2];
  unsigned char half;
  unsigned char pad_[2];
};
static_assert(sizeof(PairTile) == 16, "PairTile is read as one 16-byte entry");

// Parameters of one launch of the Newton-Schulz GEMM kernel.  Each output
// element is  scale * (c_acc * acc + c_in * in) + diag_add * [row == col].
struct GemmParams {
  CUtensorMap map_a;      // operand A, K-major: box {64 K, 128 rows}, 128B swizzle
  CUtensorMap map_a64;    // operand A, MN-major (transposed read of a symmetric matrix stored
                          // as its upper blocks): box {64 rows, 64 K}, 128B swizzle
  CUtensorMap map_b;      // operand B: box {64, 64}, 128B swizzle (K-major: {K, rows};
                          // MN-major: {N, K})
  CUtensorMap map_in;     // epilogue input, box {64, 32}, 128B swizzle
  CUtensorMap map_out;    // output (and the O tap of the last iteration), box {64, 32}, 128B swizzle
  const CUtensorMap* wmaps;  // last iteration: one map per matrix over its W (chunk-relative),
                             // box {64, 32}, 128B swizzle
  const PairTile* tiles;    // tile table of one unit of `unit_mats` consecutive matrices
  const PairTile* tiles_tail;  // unit_mats == 2 and an odd count: table of the last matrix alone
  const PairTile* tiles_t;  // last iteration: table of a matrix stored with rows > cols, whose
                            // product is formed transposed (row pairs along the long side)
  int tiles_per_unit;
  int tiles_per_tail;
  int unit_mats;   // 1, or 2 where the table pairs blocks of two matrices in one tile
  int count;       // matrices in this launch
  int k;           // contraction length
  int m;           // output rows per matrix (short side of the bucket)
  int n_long;      // long side of the bucket (output rows of a transposed-formulation tile)
  int out_cols;    // output columns per matrix
  int a_sym;       // operand A is a symmetric matrix kept as its 128-blocks on or above the
                   // diagonal: blocks below it are read as the transposes of their mirror images
  int b_sym;       // the same for operand B
  int b_mn_major;  // operand B is read MN-major throughout (X in X' = a X + B X)
  int has_in;      // the epilogue reads an input tile through map_in
  int scale_kind;  // 0: none, 1: s^2 of the matrix, 2: s
  int last;        // fused weight update: W is read, updated and written back
  int w_fp32;      // last: the weights are fp32 (maps of box {32, 32}), else bf16 (box {64, 32})
  float c_acc, c_in, diag_add;
  float upd_scale, decay;
  const MatDesc* descs;
  const MatScal* scal;
  DevStatus* status;
  float* rms_partials;  // last iteration: sums of O^2, [matrix][tile][CTA of the pair][epilogue warp]
  unsigned* debug;  // optional: TMEM base addresses seen by each CTA (test tap)
};

struct StreamParams {
  const MatDesc* descs;
  float* partials;  // [count][tiles_per_matrix]
  __nv_bfloat16* x;    // [count][m][ldx], short side first
  long long x_stride;  // elements per matrix
  int ldx;
  int count;
  int tiles_per_matrix;
  float mu;
  int nesterov;
  const int* g_bad;  // optional: per matrix, non-zero = its gradient is non-finite, leave M as it is
};

// Parameters of the TMA-pipelined momentum kernel (64 x 64 tiles).
struct StreamTmaParams {
  CUtensorMap map_x;         // bf16 X buffer [count][m][ldx], box {64, 64}, 128B swizzle
  const CUtensorMap* gmaps;  // per matrix (chunk-relative): G, box {64, 64}, no swizzle
  const CUtensorMap* mmaps;  // per matrix: M (fp32), box {64, 64}, no swizzle
  const MatDesc* descs;
  float* partials;           // [count][tiles_per_matrix]
  DevStatus* status;
  int count;
  int tiles_per_matrix;      // ceil(m / 64) * ceil(n / 64)
  int m, n;                  // short and long side of the bucket
  float mu;
  int nesterov;
  const int* g_bad;          // optional: per matrix, non-zero = its gradient is non-finite, leave M as it is
};

}  // namespace muon
