// Host side of the Muon step library: descriptor validation, shape-bucket
// planner, workspace carving, TMA descriptor encoding, launch sequencing and
// the C ABI declared in include/muon.h.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/muon.h"
#include "internal.h"

namespace muon {

cudaError_t launch_momentum_cast(const StreamParams& P, bool grad_fp32, cudaStream_t stream);
cudaError_t launch_grad_finite(const MatDesc* descs, int count, int rows_max, bool grad_fp32, int* bad,
                               cudaStream_t stream);
cudaError_t launch_norm_finalise(const float* partials, int tiles_per_matrix, int count, float eps,
                                 const MatDesc* descs, MatScal* scal, float* norms, DevStatus* status,
                                 cudaStream_t stream);
cudaError_t launch_update_from_x(const MatDesc* descs, const MatScal* scal, const float* factors,
                                 const __nv_bfloat16* x, long long x_stride, int ldx, int count, int m,
                                 int n, float neg_lr, float decay, bool w_fp32, cudaStream_t stream);
cudaError_t launch_rms_finalise(const float* partials, int per_matrix, int count, float factor,
                                const MatDesc* descs, const MatScal* scal, bool use_inv_norm, float rms_target,
                                bool normalise, float* rms, float* factors, cudaStream_t stream);
cudaError_t launch_symmetrise_diag(__nv_bfloat16* s, long long stride, int lda, int m, int count,
                                   cudaStream_t stream);
cudaError_t launch_sumsq_x(const __nv_bfloat16* x, long long x_stride, int ldx, int m, int n, int count,
                           int per_matrix, float* partials, cudaStream_t stream);
cudaError_t stream_tma_configure();
cudaError_t launch_momentum_tma(const StreamTmaParams& P, bool grad_fp32, int num_sms, cudaStream_t stream);
cudaError_t launch_wait_expiry_probe(DevStatus* status, int matrix_index, unsigned long long limit_ns,
                                     cudaStream_t stream);
cudaError_t gemm_configure();
cudaError_t gemm_max_clusters(int* out);
cudaError_t launch_ns_gemm(const GemmParams& P, int acc_cols, int max_clusters, cudaStream_t stream);

namespace {

thread_local std::string g_last_error;
int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  g_last_error = buf;
  return code;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Upper bound on the Newton-Schulz operand bytes of one chunk; larger buckets
// are processed in several chunks that reuse the same workspace.
constexpr size_t kChunkBytesDefault = size_t(8) << 30;
size_t g_chunk_bytes_max = kChunkBytesDefault;  // process-wide; see muon_debug_set_chunk_bytes
constexpr int kChunkCountMax = 4096;
// Gradient bytes per slice of the host-buffer step (muon_step_host).
#ifndef MUON_HOST_SLICE_BYTES
#define MUON_HOST_SLICE_BYTES (size_t(32) << 20)
#endif
constexpr size_t kHostSliceBytes = MUON_HOST_SLICE_BYTES;

// Two iterations per pass over X.  With P_k = a*I + b*A_k + c*A_k^2 (symmetric, a
// polynomial in A_k = X_k X_k^T) Eq. 2 reads X_{k+1} = P_k X_k, hence
//   A_{k+1} = P_k A_k P_k = P_k^2 A_k   and   X_{k+2} = (P_{k+1} P_k) X_k:
// the Gram product and the combine (m^2 n each way) of the second iteration
// are replaced by three more symmetric m x m x m products, 3 m^2 n + 5 m^3
// instead of 6 m^2 n + 2 m^3 for the two iterations, which pays when the long
// side is above the short side.
// By default only the first two iterations are taken as a pair: with bf16
// storage that is as close to the exact iteration as the plain sequence from
// 256 rows on, for every spectrum tried on a CPU model (closer for spectra with
// a wide range, where rounding X_1 to bf16 is what loses the small singular
// values).  Later pairs work near the band, where the terms of P nearly cancel:
// they cost accuracy (up to twice the plain sequence's distance on decaying
// spectra) and are only taken on request (pair-fold mode 3).
constexpr int kFoldIdentityMinRows = 16;  // from here on B' = B + a*I is kept and the combine is B' X
constexpr int kPairFoldMinRows = 256;
constexpr double kPairFirstMinAspect = 1.25;
constexpr double kPairAllMinAspect = 2.0;
// 0: first pair by shape, 1: never, 2: first pair whenever a*I is folded,
// 3: every pair by shape, 4: every pair whenever a*I is folded; see muon_debug_set_pair_fold
int g_pair_fold_mode = 0;

// How many leading pairs of `ns_steps` iterations are taken two per pass in pair-fold mode `mode`.
int plan_pairs(int mode, int m, int n, bool fold_identity, int ns_steps) {
  if (!fold_identity || mode == 1 || ns_steps < 2) return 0;
  const bool big = m >= kPairFoldMinRows;
  switch (mode) {
    case 0: return big && n >= kPairFirstMinAspect * m ? 1 : 0;
    case 2: return 1;
    case 3: return big && n >= kPairAllMinAspect * m ? ns_steps / 2 : (big && n >= kPairFirstMinAspect * m ? 1 : 0);
    case 4: return ns_steps / 2;
    default: return 0;
  }
}

struct MatRef {
  int group, index, global;
};

struct Bucket {
  int m, n;  // short side, long side
  int w_dtype, g_dtype;
  std::vector<MatRef> mats;
  int chunk;        // matrices per chunk
  int ldx, lda;
  size_t x_stride, a_stride;  // elements per matrix
  int stream_tiles;           // per-matrix partial sums reserved for the streaming kernels
  int stream_tiles_generic;   // tiles per matrix of the generic streaming kernel (64 x 128)
  int stream_tiles_tma;       // tiles per matrix of the TMA streaming kernel (64 x 64)
  bool fused_update;          // every W (and bf16 copy) is TMA-addressable: update W in the last epilogue
  bool stream_tma;            // every G and M is TMA-addressable: TMA-pipelined momentum kernel
  bool fold_identity;         // keep B' = B + a*I so that the combine is the single product B' X
  bool pair_fold;             // some iterations are taken two per pass over X (see plan_pairs)
  int pair_mode;              // the pair-fold mode the plan was made with
  // workspace offsets (bytes) of the chunk buffers
  // off_s: the symmetric m x m buffers (A and B; two more when iterations are taken in pairs)
  size_t off_x[2], off_s[4], off_partials, off_scal, off_rms_partials, off_factors, off_bad;
  // workspace offsets of the persistent per-bucket tables
  size_t off_descs, off_wmaps, off_gmaps, off_mmaps, off_sym_tiles, off_sym_tiles_tail, off_comb_tiles, off_comb_tiles_t;
  std::vector<PairTile> sym_tiles;       // symmetric products: table of one unit of sym_unit_mats matrices
  std::vector<PairTile> sym_tiles_tail;  // sym_unit_mats == 2: table of a last matrix without a partner
  int sym_unit_mats;
  std::vector<PairTile> comb_tiles;      // combine: table of one matrix
  std::vector<PairTile> comb_tiles_t;    // combine formed transposed: row pairs along the long side
  int sym_acc_cols, comb_acc_cols;       // widest tile of each table (128 or 256)
  // tensor maps over the chunk buffers (all 128-byte swizzled)
  CUtensorMap x_op[2];   // X as K-major operand A: box {64,128}
  CUtensorMap x_b64[2];  // X as operand B (K-major or MN-major): box {64,64}
  CUtensorMap x_e[2];    // X as epilogue input / output: box {64,32}
  CUtensorMap s_op[4];   // symmetric buffer as K-major operand A: box {64,128}
  CUtensorMap s_b64[4];  // as operand B or as transposed (MN-major) operand A: box {64,64}
  CUtensorMap s_e[4];    // as epilogue input / output: box {64,32}
};

struct PlanSizes {
  size_t total;
  size_t off_status;
  size_t off_norms;  // float per matrix (global order)
  size_t off_rms;    // float per matrix: update RMS of the last step
  size_t off_debug;  // TMEM base addresses seen by the CTAs of the GEMM kernel
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess) {
    return nullptr;
  }
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// 3-D bf16 map over [count][rows][cols] with row pitch `ld` elements.
int encode_map(CUtensorMap* out, void* base, int cols, int rows, int count, int ld,
               size_t mat_stride_elems, int box_x, int box_y, bool swizzle128) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows),
                        static_cast<cuuint64_t>(count)};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * 2, static_cast<cuuint64_t>(mat_stride_elems) * 2};
  cuuint32_t box[3] = {static_cast<cuuint32_t>(box_x), static_cast<cuuint32_t>(box_y), 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return MUON_OK;
}

// Map over one caller-owned matrix [rows][cols] of bf16 or fp32 with row pitch
// ld elements: box {64, 64}, not swizzled (tiles of the streaming kernel).
int encode_stream_map(CUtensorMap* out, const void* base, int rows, int cols, long long ld, bool fp32) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  const cuuint64_t es = fp32 ? 4 : 2;
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), 1};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * es, static_cast<cuuint64_t>(ld) * es * rows};
  cuuint32_t box[3] = {64, 64, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return MUON_OK;
}

// Map over one caller-owned bf16 weight matrix [rows][cols] with row pitch ld.
// The last epilogue produces its tiles in W's own orientation, so one box shape
// serves both orientations: {64, 32}, 128-byte swizzle.
int encode_w_map(CUtensorMap* out, void* w, int rows, int cols, long long ld) {
  return encode_map(out, w, cols, rows, 1, static_cast<int>(ld), static_cast<size_t>(rows) * ld, 64, 32, true);
}

// The same for an fp32 weight matrix: a 128-byte swizzled row holds 32 columns,
// so the box is {32, 32} and a 64-column quarter of the epilogue takes two.
int encode_w_map_fp32(CUtensorMap* out, void* w, int rows, int cols, long long ld) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), 1};
  cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * 4, static_cast<cuuint64_t>(ld) * 4 * rows};
  cuuint32_t box[3] = {32, 32, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, w, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(MUON_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return MUON_OK;
}

int validate_groups(const muon_group* groups, int n_groups, bool need_ptrs) {
  if (!groups || n_groups <= 0) return fail(MUON_ERR_INVALID_ARG, "groups is null or n_groups <= 0");
  for (int g = 0; g < n_groups; ++g) {
    const muon_group& G = groups[g];
    if (G.rows <= 0 || G.cols <= 0 || G.count <= 0)
      return fail(MUON_ERR_INVALID_ARG, "group %d: rows, cols and count must be positive", g);
    if (G.rows > 65536 || G.cols > 65536)
      return fail(MUON_ERR_UNSUPPORTED, "group %d: dimensions above 65536 are not supported", g);
    if ((G.w_dtype != MUON_DTYPE_BF16 && G.w_dtype != MUON_DTYPE_FP32) ||
        (G.g_dtype != MUON_DTYPE_BF16 && G.g_dtype != MUON_DTYPE_FP32))
      return fail(MUON_ERR_UNSUPPORTED, "group %d: dtype must be bf16 or fp32", g);
    if (!need_ptrs) continue;
    if (!G.w || !G.g || !G.m) return fail(MUON_ERR_INVALID_ARG, "group %d: null pointer array", g);
    if (G.ld_w < G.cols || G.ld_g < G.cols || G.ld_m < G.cols)
      return fail(MUON_ERR_INVALID_ARG, "group %d: leading dimension smaller than cols", g);
    for (int i = 0; i < G.count; ++i) {
      if (!G.w[i] || !G.g[i] || !G.m[i])
        return fail(MUON_ERR_INVALID_ARG, "group %d matrix %d: null device pointer", g, i);
      const uintptr_t wa = G.w_dtype == MUON_DTYPE_FP32 ? 3 : 1, ga = G.g_dtype == MUON_DTYPE_FP32 ? 3 : 1;
      if ((reinterpret_cast<uintptr_t>(G.w[i]) & wa) || (reinterpret_cast<uintptr_t>(G.g[i]) & ga) ||
          (reinterpret_cast<uintptr_t>(G.m[i]) & 3))
        return fail(MUON_ERR_ALIGNMENT, "group %d matrix %d: pointer not aligned to its element size", g, i);
      if (G.w[i] == G.g[i] || G.w[i] == (void*)G.m[i] || G.g[i] == (const void*)G.m[i])
        return fail(MUON_ERR_INVALID_ARG, "group %d matrix %d: W, G and M must not alias", g, i);
      if (G.w_shadow) {
        if (G.w_dtype != MUON_DTYPE_FP32)
          return fail(MUON_ERR_INVALID_ARG, "group %d: a bf16 shadow copy needs fp32 weights", g);
        if (!G.w_shadow[i] || (reinterpret_cast<uintptr_t>(G.w_shadow[i]) & 1) || G.ld_shadow < G.cols)
          return fail(MUON_ERR_INVALID_ARG, "group %d matrix %d: bad shadow pointer or leading dimension", g, i);
        if (G.w_shadow[i] == G.w[i] || G.w_shadow[i] == G.g[i] || G.w_shadow[i] == (void*)G.m[i])
          return fail(MUON_ERR_INVALID_ARG, "group %d matrix %d: the shadow copy must not alias W, G or M", g, i);
      }
    }
  }
  return MUON_OK;
}

// True if a weight matrix can be addressed by a TMA descriptor (16-byte aligned
// base and row pitch).
inline bool w_tma_ok(const void* w, long long ld, bool fp32) {
  return (reinterpret_cast<uintptr_t>(w) & 15) == 0 && ld % (fp32 ? 4 : 8) == 0;
}

PairTile make_tile(int i0, int i1, int j0, int j1, int nbw, int dm0, int dm1, unsigned keep0, unsigned keep1) {
  PairTile t{};
  t.i[0] = static_cast<short>(i0);
  t.i[1] = static_cast<short>(i1);
  t.j[0] = static_cast<short>(j0);
  t.j[1] = static_cast<short>(j1);
  t.nbw = static_cast<unsigned char>(nbw);
  t.dm[0] = static_cast<unsigned char>(dm0);
  t.dm[1] = static_cast<unsigned char>(dm1);
  t.keep[0] = static_cast<unsigned char>(keep0);
  t.keep[1] = static_cast<unsigned char>(keep1);
  return t;
}

// A half-height tile: row block i alone (64 rows in each CTA) against column blocks j0 (, j1).
PairTile make_half_tile(int i, int j0, int j1, int nbw, int dm, unsigned keep) {
  PairTile t = make_tile(i, i, j0, j1, nbw, dm, dm, keep, 0u);
  t.half = 1;
  return t;
}

// How tiles are cut where the row blocks do not pair up; see muon_debug_set_tile_mode.
// bit 0: a row block without a partner is taken at half height; bit 1: so is a lone diagonal block;
// bit 2: launches with few tiles are NOT cut finer.
// Measured on the expert bucket (1408 rows = 11 row blocks): mode 1 13.49 ms per step, mode 0 13.67,
// mode 3 13.67, mode 2 13.83: the half-height, half-width tiles of bit 1 run too far below the
// tensor cores' rate to pay, although they compute nothing in vain.
int g_tile_mode = 1;
constexpr int kNominalPairs = 74;  // CTA pairs of a B200 (148 SMs); a planning constant, not a device query

// Tiles of the symmetric products (only the 128-blocks on or above the diagonal
// are produced) for matrix `dm` of a unit, nb row blocks.  A full tile is two
// neighbouring row blocks times two neighbouring column blocks.  Row pair
// (r, r+1), r even, takes the columns from r+1 on two at a time (a last single
// column as a tile of half the width); every block of these tiles is kept.  That
// leaves the diagonal blocks (r, r), r even, which no full tile can hold without
// waste (the block below it in the pair lies under the diagonal): with
// `half_lone` each becomes a half-height, half-width tile, otherwise `lone`
// receives them (an odd number of row blocks; an even number needs none, see below).
void sym_tiles_of_matrix(int nb, int dm, bool half_lone, std::vector<PairTile>* tiles, std::vector<int>* lone) {
  if (nb % 2 == 0 && !half_lone) {
    // an even number of row blocks: row pair (r, r+1) takes columns r, r+1, then r+2, r+3, ...: every
    // tile is full width; the first holds the block (r+1, r) under the diagonal, computed and dropped
    // (nb/2 blocks in nb(nb+1)/2 + nb/2), which is cheaper than half-width tiles at the end of every row pair
    for (int r = 0; r < nb; r += 2)
      for (int c = r; c < nb; c += 2)
        tiles->push_back(make_tile(r, r + 1, c, c + 1, 2, dm, dm, 3u, c == r ? 2u : 3u));
    return;
  }
  for (int r = 0; r < nb; r += 2) {
    if (half_lone) tiles->push_back(make_half_tile(r, r, r, 1, dm, 1u));
    else lone->push_back(r);
    if (r + 1 >= nb) break;
    for (int c = r + 1; c < nb; c += 2) {
      const int w = std::min(2, nb - c);
      tiles->push_back(make_tile(r, r + 1, c, c + 1, w, dm, dm, w == 2 ? 3u : 1u, w == 2 ? 3u : 1u));
    }
  }
}

// Tile tables of a bucket.
void build_tile_tables(Bucket* Bp) {
  Bucket& B = *Bp;
  const int nb = ceil_div(B.m, 128), ncb = ceil_div(B.n, 128), np = ceil_div(nb, 2);
  const bool half_rows = (g_tile_mode & 1) != 0, half_lone = (g_tile_mode & 2) != 0;
  B.sym_tiles.clear();
  B.sym_tiles_tail.clear();
  B.comb_tiles.clear();
  B.comb_tiles_t.clear();
  B.sym_acc_cols = B.comb_acc_cols = 128;
  std::vector<int> lone;
  if (half_lone || nb % 2 == 0) {
    B.sym_unit_mats = 1;
    sym_tiles_of_matrix(nb, 0, half_lone, &B.sym_tiles, &lone);
  } else {
    // Without half-height tiles the lone diagonal blocks (r, r) of two matrices share a
    // full-width tile, one CTA per matrix, whose two cross blocks are dropped; a matrix
    // alone takes each with the block below it, which lies under the diagonal and is dropped.
    B.sym_unit_mats = 2;
    sym_tiles_of_matrix(nb, 0, false, &B.sym_tiles, &lone);
    lone.clear();
    sym_tiles_of_matrix(nb, 1, false, &B.sym_tiles, &lone);
    for (int r : lone) B.sym_tiles.push_back(make_tile(r, r, r, r, 2, 0, 1, 1u, 2u));
    lone.clear();
    sym_tiles_of_matrix(nb, 0, false, &B.sym_tiles_tail, &lone);
    for (int r : lone) B.sym_tiles_tail.push_back(make_tile(r, r + 1, r, r, 1, 0, 0, 1u, 0u));
  }
  // A launch with fewer tiles than CTA pairs leaves SMs idle: a bucket of few small matrices is then
  // cut finer, every row block on its own at half height (twice the tiles at about 0.6 of a full tile's
  // time each), or block by block (four times the tiles at about 0.45).  The estimate is rounds of
  // kNominalPairs concurrent tiles times the tile's relative time; full tiles win whenever the SMs are busy.
  {
    const int count = std::max(1, std::min<int>(B.chunk > 0 ? B.chunk : 1, static_cast<int>(B.mats.size())));
    const long long t_full = static_cast<long long>(count / B.sym_unit_mats) * static_cast<long long>(B.sym_tiles.size()) +
                             (count % B.sym_unit_mats) * static_cast<long long>(B.sym_tiles_tail.size());
    long long t_rows = 0;
    for (int i = 0; i < nb; ++i) t_rows += ceil_div(nb - i, 2);
    t_rows *= count;
    const long long t_blocks = static_cast<long long>(count) * nb * (nb + 1) / 2;
    auto rounds = [](long long t) { return static_cast<double>((t + kNominalPairs - 1) / kNominalPairs); };
    const double c_full = rounds(t_full) * 1.0, c_rows = rounds(t_rows) * 0.6, c_blocks = rounds(t_blocks) * 0.45;
    if ((g_tile_mode & 4) == 0 && t_full < kNominalPairs && (c_rows < c_full || c_blocks < c_full)) {
      const bool by_block = c_blocks < c_rows;
      B.sym_tiles.clear();
      B.sym_tiles_tail.clear();
      B.sym_unit_mats = 1;
      for (int i = 0; i < nb; ++i)
        for (int c = i; c < nb;) {
          const int w = by_block ? 1 : std::min(2, nb - c);
          B.sym_tiles.push_back(make_half_tile(i, c, c + 1, w, 0, w == 2 ? 3u : 1u));
          c += w;
        }
    }
  }
  for (const PairTile& t : B.sym_tiles)
    if (t.nbw == 2) B.sym_acc_cols = 256;
  // combine: row pair p covers row blocks 2p, 2p+1 (a last row block without a partner
  // at half height); column tiles are two 128-blocks wide, with one single block at the
  // end of an odd run
  auto rows_by_cols = [&](int row_blocks, int col_blocks, std::vector<PairTile>* out) {
    for (int p = 0; p < ceil_div(row_blocks, 2); ++p) {
      const bool single = 2 * p + 1 >= row_blocks && half_rows;
      for (int jb = 0; jb < col_blocks;) {
        const int w = std::min(2, col_blocks - jb);
        if (single) out->push_back(make_half_tile(2 * p, jb, jb + 1, w, 0, w == 2 ? 3u : 1u));
        else out->push_back(make_tile(2 * p, 2 * p + 1, jb, jb + 1, w, 0, 0, w == 2 ? 3u : 1u, w == 2 ? 3u : 1u));
        jb += w;
      }
    }
  };
  rows_by_cols(nb, ncb, &B.comb_tiles);
  if (ncb >= 2) B.comb_acc_cols = 256;
  // the same product with the roles of the sides exchanged (as many tiles)
  rows_by_cols(ncb, nb, &B.comb_tiles_t);
  (void)np;
}

// Forms the shape buckets and lays out the workspace.  Deterministic in the
// group list (pointers are not consulted), so muon_workspace_bytes and
// muon_init agree.
int make_plan(const muon_group* groups, int n_groups, std::vector<Bucket>* buckets, PlanSizes* sizes,
              int* total_mats) {
  std::map<std::tuple<int, int, int, int>, int> index;
  buckets->clear();
  int global = 0;
  for (int g = 0; g < n_groups; ++g) {
    const muon_group& G = groups[g];
    const int m = std::min(G.rows, G.cols), n = std::max(G.rows, G.cols);
    auto key = std::make_tuple(m, n, G.w_dtype, G.g_dtype);
    auto it = index.find(key);
    int b;
    if (it == index.end()) {
      b = static_cast<int>(buckets->size());
      index[key] = b;
      Bucket nb{};
      nb.m = m;
      nb.n = n;
      nb.w_dtype = G.w_dtype;
      nb.g_dtype = G.g_dtype;
      buckets->push_back(nb);
    } else {
      b = it->second;
    }
    for (int i = 0; i < G.count; ++i) (*buckets)[b].mats.push_back(MatRef{g, i, global++});
  }
  *total_mats = global;

  // Chunk buffers are shared by all buckets (they run one after another), so
  // the workspace is the maximum over buckets, not the sum.
  size_t chunk_region = 0;
  for (Bucket& B : *buckets) {
    B.ldx = static_cast<int>(align_up(B.n, 64));
    B.lda = static_cast<int>(align_up(B.m, 64));
    B.x_stride = static_cast<size_t>(B.m) * B.ldx;
    B.a_stride = static_cast<size_t>(B.m) * B.lda;
    // tile counts of the streaming kernel for both stored orientations
    const int t1 = ceil_div(B.m, kSTR) * ceil_div(B.n, kSTC);
    const int t2 = ceil_div(B.n, kSTR) * ceil_div(B.m, kSTC);
    B.stream_tiles_generic = std::max(t1, t2);
    B.stream_tiles_tma = ceil_div(B.m, 64) * ceil_div(B.n, 64);
    B.stream_tiles = std::max(B.stream_tiles_generic, B.stream_tiles_tma);
    // Folding a*X into the product rounds B_ii + a to bf16; that is the smaller
    // error from 16 rows up (measured with a bf16 storage model) and the larger one below.
    B.fold_identity = B.m >= kFoldIdentityMinRows;
    B.pair_fold = plan_pairs(g_pair_fold_mode, B.m, B.n, B.fold_identity, 64) > 0;
    B.pair_mode = g_pair_fold_mode;
    const int n_sym = B.pair_fold ? 4 : 2;
    const size_t per_mat = 2 * B.x_stride * 2 + n_sym * B.a_stride * 2;
    size_t chunk = std::max<size_t>(1, g_chunk_bytes_max / per_mat);
    chunk = std::min<size_t>(chunk, B.mats.size());
    chunk = std::min<size_t>(chunk, kChunkCountMax);
    // keep the streaming grid within 2^31 CTAs
    while (chunk > 1 && chunk * static_cast<size_t>(B.stream_tiles) > (size_t(1) << 30)) chunk /= 2;
    B.chunk = static_cast<int>(chunk);
    size_t off = 0;
    auto take = [&off](size_t bytes) {
      size_t o = off;
      off = align_up(off + bytes, 1024);
      return o;
    };
    B.off_x[0] = take(chunk * B.x_stride * 2);
    B.off_x[1] = take(chunk * B.x_stride * 2);
    for (int i = 0; i < 4; ++i) B.off_s[i] = i < n_sym ? take(chunk * B.a_stride * 2) : 0;
    B.off_partials = take(chunk * static_cast<size_t>(B.stream_tiles) * sizeof(float));
    B.off_scal = take(chunk * sizeof(MatScal));
    // sums of O^2 of the last epilogue: per matrix, comb tile, CTA of the pair and epilogue warp
    {
      const int ncb = ceil_div(B.n, 128), np = ceil_div(ceil_div(B.m, 128), 2);
      const size_t comb_tiles = static_cast<size_t>(np) * ceil_div(ncb, 2);
      B.off_rms_partials = take(chunk * comb_tiles * 8 * sizeof(float));
    }
    B.off_factors = take(chunk * sizeof(float));
    B.off_bad = take(chunk * sizeof(int));
    chunk_region = std::max(chunk_region, off);
  }
  size_t off = align_up(chunk_region, 1024);
  // persistent region: descriptors and W maps of every matrix (bucket by bucket),
  // tile tables, status, norms
  for (Bucket& B : *buckets) {
    B.off_descs = off;
    off = align_up(off + B.mats.size() * sizeof(MatDesc), 1024);
    B.off_wmaps = off;
    off = align_up(off + B.mats.size() * sizeof(CUtensorMap), 1024);
    B.off_gmaps = off;
    off = align_up(off + B.mats.size() * sizeof(CUtensorMap), 1024);
    B.off_mmaps = off;
    off = align_up(off + B.mats.size() * sizeof(CUtensorMap), 1024);
    build_tile_tables(&B);
    B.off_sym_tiles = off;
    off = align_up(off + B.sym_tiles.size() * sizeof(PairTile), 1024);
    B.off_sym_tiles_tail = off;
    off = align_up(off + B.sym_tiles_tail.size() * sizeof(PairTile), 1024);
    B.off_comb_tiles = off;
    off = align_up(off + B.comb_tiles.size() * sizeof(PairTile), 1024);
    B.off_comb_tiles_t = off;
    off = align_up(off + B.comb_tiles_t.size() * sizeof(PairTile), 1024);
  }
  sizes->off_debug = off;
  off = align_up(off + 1024 * sizeof(unsigned), 1024);
  sizes->off_status = off;
  off = align_up(off + sizeof(DevStatus), 1024);
  sizes->off_norms = off;
  off = align_up(off + static_cast<size_t>(global) * sizeof(float), 1024);
  sizes->off_rms = off;
  off = align_up(off + static_cast<size_t>(global) * sizeof(float), 1024);
  sizes->total = off;
  return MUON_OK;
}

}  // namespace

// Lets the other translation units of the library report through muon_last_error().
void set_last_error(const char* msg) { g_last_error = msg ? msg : ""; }

}  // namespace muon

using namespace muon;

struct muon_ctx {
  int device;
  int num_sms;
  int max_clusters;  // co-resident CTA pairs of the GEMM kernel
  int keep_o;
  int last_launches;
  uint8_t* ws;
  size_t ws_bytes;
  std::vector<muon_group> groups;            // copies (pointer arrays re-owned below)
  std::vector<std::vector<void*>> w_ptrs;    // per group
  std::vector<std::vector<const void*>> g_ptrs;
  std::vector<std::vector<float*>> m_ptrs;
  std::vector<std::vector<void*>> s_ptrs;    // optional bf16 shadow copies
  std::vector<Bucket> buckets;
  PlanSizes sizes;
  int total_mats;
  // where each global matrix lives: bucket and position
  std::vector<std::pair<int, int>> where;
  // debug taps: which X buffer holds X0 / the last X per bucket
  std::vector<int> x0_buf, xlast_buf;
  std::vector<int> a_last_buf, b_last_buf;  // symmetric buffers holding the last iteration's A and B
  // per-launch timing (measurement mode)
  int profile;
  std::vector<cudaEvent_t> ev_pool;           // pairs: start, stop
  std::vector<int> ev_kind;                   // kind of each recorded pair
  size_t ev_used;
  // host-buffer path: copy streams and the events that order copies and kernels
  cudaStream_t s_in = nullptr, s_out = nullptr;
  std::vector<cudaEvent_t> pipe_events;
  ~muon_ctx() {
    for (cudaEvent_t e : ev_pool) cudaEventDestroy(e);
    for (cudaEvent_t e : pipe_events) cudaEventDestroy(e);
    if (s_in) cudaStreamDestroy(s_in);
    if (s_out) cudaStreamDestroy(s_out);
  }
};

namespace {
// Makes the context's device current for the duration of a call and restores
// the caller's device afterwards (launches and copies go to the current device).
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int device) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != device) switched = (cudaSetDevice(device) == cudaSuccess);
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

// Records an event pair around one launch when the context is in measurement mode.
struct LaunchTimer {
  muon_ctx* ctx;
  cudaStream_t stream;
  bool on;
  LaunchTimer(muon_ctx* c, cudaStream_t s, int kind) : ctx(c), stream(s), on(c->profile != 0) {
    if (!on) return;
    if (ctx->ev_used + 2 > ctx->ev_pool.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
      ctx->ev_pool.push_back(a);
      ctx->ev_pool.push_back(b);
    }
    ctx->ev_kind.push_back(kind);
    cudaEventRecord(ctx->ev_pool[ctx->ev_used], stream);
  }
  ~LaunchTimer() {
    if (!on) return;
    cudaEventRecord(ctx->ev_pool[ctx->ev_used + 1], stream);
    ctx->ev_used += 2;
  }
};
}  // namespace

extern "C" {

const char* muon_last_error(void) { return g_last_error.c_str(); }

size_t muon_debug_set_chunk_bytes(size_t bytes) {
  const size_t prev = g_chunk_bytes_max;
  g_chunk_bytes_max = bytes ? bytes : kChunkBytesDefault;
  return prev;
}

int muon_partition(const muon_group* groups, int n_groups, int world, int* owner_out, double* load_out) {
  if (!owner_out || world <= 0) return fail(MUON_ERR_INVALID_ARG, "owner_out is null or world <= 0");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  // cost of one matrix: the Newton-Schulz work per iteration, 3 m^2 n + m^3
  struct Item { double cost; int global; };
  std::vector<Item> items;
  int global = 0;
  for (int g = 0; g < n_groups; ++g) {
    const double m = std::min(groups[g].rows, groups[g].cols), n = std::max(groups[g].rows, groups[g].cols);
    const double cost = 3.0 * m * m * n + m * m * m;
    for (int i = 0; i < groups[g].count; ++i) items.push_back(Item{cost, global++});
  }
  // longest processing time first: heaviest matrices first, each to the least
  // loaded rank; ties by matrix order and by rank, so every rank computes the
  // same assignment
  std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) { return a.cost > b.cost; });
  std::vector<double> load(world, 0.0);
  for (const Item& it : items) {
    int best = 0;
    for (int r = 1; r < world; ++r)
      if (load[r] < load[best]) best = r;
    owner_out[it.global] = best;
    load[best] += it.cost;
  }
  if (load_out)
    for (int r = 0; r < world; ++r) load_out[r] = load[r];
  return MUON_OK;
}

int muon_partition_slots(const muon_group* groups, int n_groups, int world, int* owner_out, int* pos_out,
                         int* share_out, double* load_out) {
  if (!owner_out || !pos_out || !share_out || world <= 0)
    return fail(MUON_ERR_INVALID_ARG, "an output pointer is null or world <= 0");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  std::vector<Bucket> buckets;
  PlanSizes sizes;
  int total;
  rc = make_plan(groups, n_groups, &buckets, &sizes, &total);
  if (rc) return rc;
  std::vector<double> load(world, 0.0);
  std::vector<int> order(world);
  for (size_t b = 0; b < buckets.size(); ++b) {
    const Bucket& B = buckets[b];
    const int cnt = static_cast<int>(B.mats.size());
    const double m = B.m, n = B.n, cost = 3.0 * m * m * n + m * m * m;
    const int base = cnt / world, extra = cnt % world;
    share_out[b] = base + (extra ? 1 : 0);
    // the `extra` ranks with one matrix more are the least loaded so far (ties: lower rank)
    for (int r = 0; r < world; ++r) order[r] = r;
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return load[x] < load[y]; });
    std::vector<int> mine(world, base);
    for (int k = 0; k < extra; ++k) mine[order[k]] += 1;
    // consecutive runs of the bucket's matrices, rank by rank
    int next = 0;
    for (int r = 0; r < world; ++r) {
      for (int k = 0; k < mine[r]; ++k) {
        const int g = B.mats[next++].global;
        owner_out[g] = r;
        pos_out[g] = k;
      }
      load[r] += mine[r] * cost;
    }
  }
  if (load_out)
    for (int r = 0; r < world; ++r) load_out[r] = load[r];
  return MUON_OK;
}

int muon_workspace_bytes(const muon_group* groups, int n_groups, size_t* out_bytes) {
  if (!out_bytes) return fail(MUON_ERR_INVALID_ARG, "out_bytes is null");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  std::vector<Bucket> buckets;
  PlanSizes sizes;
  int total;
  rc = make_plan(groups, n_groups, &buckets, &sizes, &total);
  if (rc) return rc;
  *out_bytes = sizes.total;
  return MUON_OK;
}

int muon_debug_set_tile_mode(int mode) {
  const int prev = g_tile_mode;
  if (mode >= 0 && mode <= 7) g_tile_mode = mode;
  return prev;
}

int muon_debug_set_pair_fold(int mode) {
  const int prev = g_pair_fold_mode;
  if (mode >= 0 && mode <= 4) g_pair_fold_mode = mode;
  return prev;
}

int muon_plan_buckets(const muon_group* groups, int n_groups, int* bucket_out, int* n_buckets_out) {
  if (!bucket_out || !n_buckets_out) return fail(MUON_ERR_INVALID_ARG, "bucket_out or n_buckets_out is null");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  std::vector<Bucket> buckets;
  PlanSizes sizes;
  int total;
  rc = make_plan(groups, n_groups, &buckets, &sizes, &total);
  if (rc) return rc;
  for (size_t b = 0; b < buckets.size(); ++b)
    for (const MatRef& r : buckets[b].mats) bucket_out[r.global] = static_cast<int>(b);
  *n_buckets_out = static_cast<int>(buckets.size());
  return MUON_OK;
}

int muon_plan_flops(const muon_group* groups, int n_groups, int ns_steps, double* algorithmic_out,
                    double* planned_out) {
  if (!algorithmic_out || !planned_out) return fail(MUON_ERR_INVALID_ARG, "output pointer is null");
  if (ns_steps < 0 || ns_steps > 64) return fail(MUON_ERR_INVALID_ARG, "ns_steps must be in [0, 64]");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  double alg = 0.0, planned = 0.0;
  for (int g = 0; g < n_groups; ++g) {
    const double m = std::min(groups[g].rows, groups[g].cols), n = std::max(groups[g].rows, groups[g].cols);
    const double one = 3.0 * m * m * n + m * m * m;     // Gram (half), polynomial (half), combine
    const double two = 3.0 * m * m * n + 5.0 * m * m * m;  // one Gram, five symmetric m^3 products, one combine
    const int n_pairs = plan_pairs(g_pair_fold_mode, static_cast<int>(m), static_cast<int>(n),
                                  m >= kFoldIdentityMinRows, ns_steps);
    alg += groups[g].count * ns_steps * one;
    planned += groups[g].count * (n_pairs * two + (ns_steps - 2 * n_pairs) * one);
  }
  *algorithmic_out = alg;
  *planned_out = planned;
  return MUON_OK;
}

int muon_plan_work(const muon_group* groups, int n_groups, int ns_steps, double* planned_by_kind,
                   double* executed_by_kind) {
  if (!planned_by_kind || !executed_by_kind) return fail(MUON_ERR_INVALID_ARG, "output pointer is null");
  if (ns_steps < 0 || ns_steps > 64) return fail(MUON_ERR_INVALID_ARG, "ns_steps must be in [0, 64]");
  int rc = validate_groups(groups, n_groups, false);
  if (rc) return rc;
  std::vector<Bucket> buckets;
  PlanSizes sizes;
  int total;
  rc = make_plan(groups, n_groups, &buckets, &sizes, &total);
  if (rc) return rc;
  for (int k = 0; k < MUON_KERNEL_KINDS; ++k) planned_by_kind[k] = executed_by_kind[k] = 0.0;
  // FLOPs one table executes: every tile is 256 rows x (128 or 256) columns x the
  // contraction length in whole 64-element pipeline stages
  auto table_flops = [](const std::vector<PairTile>& t, int k) {
    double f = 0.0;
    for (const PairTile& e : t)
      f += 2.0 * (e.half ? 128.0 : 256.0) * (128.0 * e.nbw) * (static_cast<double>(ceil_div(k, kBK)) * kBK);
    return f;
  };
  for (const Bucket& B : buckets) {
    const double m = B.m, n = B.n;
    const int n_pairs = plan_pairs(B.pair_mode, B.m, B.n, B.fold_identity, ns_steps);
    const int n_gram = ns_steps - n_pairs, n_comb = ns_steps - n_pairs;  // a pair has one of each
    const int n_poly = (ns_steps - 2 * n_pairs) + 5 * n_pairs;
    const int total_mats = static_cast<int>(B.mats.size());
    planned_by_kind[MUON_KERNEL_GRAM] += total_mats * n_gram * (m * m * n);
    planned_by_kind[MUON_KERNEL_POLY] += total_mats * n_poly * (m * m * m);
    planned_by_kind[MUON_KERNEL_COMB] += total_mats * n_comb * (2.0 * m * m * n);
    for (int first = 0; first < total_mats; first += B.chunk) {
      const int count = std::min(B.chunk, total_mats - first);
      const int units = count / B.sym_unit_mats, tail = count % B.sym_unit_mats;
      executed_by_kind[MUON_KERNEL_GRAM] +=
          n_gram * (units * table_flops(B.sym_tiles, B.n) + tail * table_flops(B.sym_tiles_tail, B.n));
      executed_by_kind[MUON_KERNEL_POLY] +=
          n_poly * (units * table_flops(B.sym_tiles, B.m) + tail * table_flops(B.sym_tiles_tail, B.m));
      // both orientations of the combine have as many tiles of the same widths
      executed_by_kind[MUON_KERNEL_COMB] += n_comb * (count * table_flops(B.comb_tiles, B.m));
    }
  }
  return MUON_OK;
}

int muon_debug_tile_table(int rows, int cols, int count, int which, int16_t* out, int cap_tiles, int* n_tiles,
                          int* unit_mats) {
  if (!n_tiles || !unit_mats || rows <= 0 || cols <= 0 || rows > 65536 || cols > 65536 || which < 0 || which > 3 ||
      count <= 0)
    return fail(MUON_ERR_INVALID_ARG, "bad arguments");
  Bucket B{};
  B.m = std::min(rows, cols);
  B.n = std::max(rows, cols);
  B.mats.resize(count);
  B.chunk = std::min(count, kChunkCountMax);
  build_tile_tables(&B);
  const std::vector<PairTile>& t = which == 0 ? B.sym_tiles : (which == 1 ? B.sym_tiles_tail : (which == 2 ? B.comb_tiles : B.comb_tiles_t));
  *n_tiles = static_cast<int>(t.size());
  *unit_mats = which == 0 ? B.sym_unit_mats : 1;
  if (out) {
    if (cap_tiles < *n_tiles) return fail(MUON_ERR_INVALID_ARG, "table has %d tiles, room for %d", *n_tiles, cap_tiles);
    for (size_t k = 0; k < t.size(); ++k) {
      int16_t* o = out + 10 * k;
      o[0] = t[k].i[0]; o[1] = t[k].i[1]; o[2] = t[k].j[0]; o[3] = t[k].j[1]; o[4] = t[k].nbw;
      o[5] = t[k].dm[0]; o[6] = t[k].dm[1]; o[7] = t[k].keep[0]; o[8] = t[k].keep[1]; o[9] = t[k].half;
    }
  }
  return MUON_OK;
}

int muon_init(muon_ctx** out_ctx, const muon_group* groups, int n_groups, void* workspace,
              size_t workspace_bytes, int device) {
  if (!out_ctx) return fail(MUON_ERR_INVALID_ARG, "out_ctx is null");
  *out_ctx = nullptr;
  int rc = validate_groups(groups, n_groups, true);
  if (rc) return rc;
  if (!workspace) return fail(MUON_ERR_WORKSPACE, "workspace is null");
  if (reinterpret_cast<uintptr_t>(workspace) & 1023)
    return fail(MUON_ERR_WORKSPACE, "workspace must be 1024-byte aligned");

  muon_ctx* ctx = new (std::nothrow) muon_ctx();
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "out of host memory");
  ctx->device = device;
  ctx->keep_o = 0;
  ctx->last_launches = 0;
  ctx->profile = 0;
  ctx->ev_used = 0;
  ctx->ws = static_cast<uint8_t*>(workspace);
  ctx->ws_bytes = workspace_bytes;
  rc = make_plan(groups, n_groups, &ctx->buckets, &ctx->sizes, &ctx->total_mats);
  if (rc) { delete ctx; return rc; }
  if (workspace_bytes < ctx->sizes.total) {
    const size_t need = ctx->sizes.total;
    delete ctx;
    return fail(MUON_ERR_WORKSPACE, "workspace too small: need %zu bytes, got %zu", need, workspace_bytes);
  }

  // `device` is current for the rest of the call; the guard restores the caller's on every return
  int caller_device = -1;
  cudaError_t ce = cudaGetDevice(&caller_device);
  if (ce == cudaSuccess) ce = cudaSetDevice(device);
  if (ce != cudaSuccess) { delete ctx; return fail(MUON_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce)); }
  struct Restore {
    int prev, cur;
    ~Restore() { if (prev >= 0 && prev != cur) cudaSetDevice(prev); }
  } restore{caller_device, device};
  cudaDeviceProp prop;
  ce = cudaGetDeviceProperties(&prop, device);
  if (ce != cudaSuccess) { delete ctx; return fail(MUON_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(ce)); }
  if (prop.major != 10) {
    delete ctx;
    return fail(MUON_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", device,
                prop.major, prop.minor);
  }
  ctx->num_sms = prop.multiProcessorCount;
  ce = gemm_configure();
  if (ce == cudaSuccess) ce = stream_tma_configure();
  if (ce == cudaSuccess) ce = gemm_max_clusters(&ctx->max_clusters);
  if (ce == cudaSuccess && ctx->max_clusters < 1) ctx->max_clusters = 1;
  if (ce != cudaSuccess) { delete ctx; return fail(MUON_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(ce)); }

  // own copies of the descriptor arrays
  ctx->groups.assign(groups, groups + n_groups);
  ctx->w_ptrs.resize(n_groups);
  ctx->g_ptrs.resize(n_groups);
  ctx->m_ptrs.resize(n_groups);
  ctx->s_ptrs.resize(n_groups);
  for (int g = 0; g < n_groups; ++g) {
    if (groups[g].w_shadow) {
      ctx->s_ptrs[g].assign(groups[g].w_shadow, groups[g].w_shadow + groups[g].count);
      ctx->groups[g].w_shadow = ctx->s_ptrs[g].data();
    }
    ctx->w_ptrs[g].assign(groups[g].w, groups[g].w + groups[g].count);
    ctx->g_ptrs[g].assign(groups[g].g, groups[g].g + groups[g].count);
    ctx->m_ptrs[g].assign(groups[g].m, groups[g].m + groups[g].count);
    ctx->groups[g].w = ctx->w_ptrs[g].data();
    ctx->groups[g].g = ctx->g_ptrs[g].data();
    ctx->groups[g].m = ctx->m_ptrs[g].data();
  }
  ctx->where.assign(ctx->total_mats, std::make_pair(-1, -1));
  ctx->x0_buf.assign(ctx->buckets.size(), 0);
  ctx->xlast_buf.assign(ctx->buckets.size(), 0);
  ctx->a_last_buf.assign(ctx->buckets.size(), 0);
  ctx->b_last_buf.assign(ctx->buckets.size(), 1);

  // per-bucket: upload matrix descriptors and W maps, encode tensor maps
  for (size_t b = 0; b < ctx->buckets.size(); ++b) {
    Bucket& B = ctx->buckets[b];
    std::vector<MatDesc> descs(B.mats.size());
    B.fused_update = true;
    const bool w_fp32 = B.w_dtype == MUON_DTYPE_FP32;
    B.stream_tma = true;
    const long long g_es = B.g_dtype == MUON_DTYPE_FP32 ? 4 : 2;
    for (size_t i = 0; i < B.mats.size(); ++i) {
      const MatRef& r = B.mats[i];
      const muon_group& G = ctx->groups[r.group];
      MatDesc d{};
      d.w = G.w[r.index];
      d.g = G.g[r.index];
      d.m = G.m[r.index];
      d.ld_w = G.ld_w;
      d.ld_g = G.ld_g;
      d.ld_m = G.ld_m;
      d.rows = G.rows;
      d.cols = G.cols;
      d.transposed = G.rows > G.cols ? 1 : 0;
      d.global_index = r.global;
      d.w_shadow = G.w_shadow ? G.w_shadow[r.index] : nullptr;
      d.ld_ws = G.ld_shadow;
      const bool ptr16 = ((reinterpret_cast<uintptr_t>(d.w) | reinterpret_cast<uintptr_t>(d.g) |
                           reinterpret_cast<uintptr_t>(d.m)) & 15) == 0;
      d.vec_ok = (ptr16 && G.ld_w % 8 == 0 && G.ld_g % 8 == 0 && G.ld_m % 8 == 0) ? 1 : 0;
      descs[i] = d;
      ctx->where[r.global] = std::make_pair(static_cast<int>(b), static_cast<int>(i));
      if (!w_tma_ok(d.w, d.ld_w, w_fp32) || d.ld_w > (1ll << 31)) B.fused_update = false;
      // the epilogue writes the bf16 copy with 16-byte stores
      if (d.w_shadow && !w_tma_ok(d.w_shadow, d.ld_ws, false)) B.fused_update = false;
      if ((reinterpret_cast<uintptr_t>(d.g) & 15) || (d.ld_g * g_es) % 16 || (reinterpret_cast<uintptr_t>(d.m) & 15) ||
          (d.ld_m * 4) % 16)
        B.stream_tma = false;
    }
    ce = cudaMemcpy(ctx->ws + B.off_descs, descs.data(), descs.size() * sizeof(MatDesc), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess)
      ce = cudaMemcpy(ctx->ws + B.off_sym_tiles, B.sym_tiles.data(), B.sym_tiles.size() * sizeof(PairTile),
                      cudaMemcpyHostToDevice);
    if (ce == cudaSuccess && !B.sym_tiles_tail.empty())
      ce = cudaMemcpy(ctx->ws + B.off_sym_tiles_tail, B.sym_tiles_tail.data(),
                      B.sym_tiles_tail.size() * sizeof(PairTile), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess)
      ce = cudaMemcpy(ctx->ws + B.off_comb_tiles, B.comb_tiles.data(), B.comb_tiles.size() * sizeof(PairTile),
                      cudaMemcpyHostToDevice);
    if (ce == cudaSuccess)
      ce = cudaMemcpy(ctx->ws + B.off_comb_tiles_t, B.comb_tiles_t.data(), B.comb_tiles_t.size() * sizeof(PairTile),
                      cudaMemcpyHostToDevice);
    if (ce == cudaSuccess && B.fused_update) {
      std::vector<CUtensorMap> wmaps(B.mats.size());
      for (size_t i = 0; i < B.mats.size() && rc == MUON_OK; ++i)
        rc = w_fp32 ? encode_w_map_fp32(&wmaps[i], descs[i].w, descs[i].rows, descs[i].cols, descs[i].ld_w)
                    : encode_w_map(&wmaps[i], descs[i].w, descs[i].rows, descs[i].cols, descs[i].ld_w);
      if (rc != MUON_OK) { delete ctx; return rc; }
      ce = cudaMemcpy(ctx->ws + B.off_wmaps, wmaps.data(), wmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice);
    }
    if (ce == cudaSuccess && B.stream_tma) {
      std::vector<CUtensorMap> gmaps(B.mats.size()), mmaps(B.mats.size());
      for (size_t i = 0; i < B.mats.size() && rc == MUON_OK; ++i) {
        rc = encode_stream_map(&gmaps[i], descs[i].g, descs[i].rows, descs[i].cols, descs[i].ld_g,
                               B.g_dtype == MUON_DTYPE_FP32);
        if (rc == MUON_OK) rc = encode_stream_map(&mmaps[i], descs[i].m, descs[i].rows, descs[i].cols, descs[i].ld_m, true);
      }
      if (rc != MUON_OK) { delete ctx; return rc; }
      ce = cudaMemcpy(ctx->ws + B.off_gmaps, gmaps.data(), gmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice);
      if (ce == cudaSuccess)
        ce = cudaMemcpy(ctx->ws + B.off_mmaps, mmaps.data(), mmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice);
    }
    if (ce != cudaSuccess) { delete ctx; return fail(MUON_ERR_CUDA, "descriptor upload: %s", cudaGetErrorString(ce)); }

    for (int p = 0; p < 2 && rc == MUON_OK; ++p) {
      void* xb = ctx->ws + B.off_x[p];
      rc = encode_map(&B.x_op[p], xb, B.n, B.m, B.chunk, B.ldx, B.x_stride, 64, 128, true);
      if (rc == MUON_OK) rc = encode_map(&B.x_b64[p], xb, B.n, B.m, B.chunk, B.ldx, B.x_stride, 64, 64, true);
      if (rc == MUON_OK) rc = encode_map(&B.x_e[p], xb, B.n, B.m, B.chunk, B.ldx, B.x_stride, 64, 32, true);
    }
    for (int i = 0; i < (B.pair_fold ? 4 : 2) && rc == MUON_OK; ++i) {
      void* sb = ctx->ws + B.off_s[i];
      rc = encode_map(&B.s_op[i], sb, B.m, B.m, B.chunk, B.lda, B.a_stride, 64, 128, true);
      if (rc == MUON_OK) rc = encode_map(&B.s_b64[i], sb, B.m, B.m, B.chunk, B.lda, B.a_stride, 64, 64, true);
      if (rc == MUON_OK) rc = encode_map(&B.s_e[i], sb, B.m, B.m, B.chunk, B.lda, B.a_stride, 64, 32, true);
    }
    if (rc != MUON_OK) { delete ctx; return rc; }
  }
  ce = cudaMemset(ctx->ws + ctx->sizes.off_status, 0, sizeof(DevStatus));
  if (ce == cudaSuccess) {
    DevStatus init{0, -1};
    ce = cudaMemcpy(ctx->ws + ctx->sizes.off_status, &init, sizeof(init), cudaMemcpyHostToDevice);
  }
  if (ce == cudaSuccess) ce = cudaMemset(ctx->ws + ctx->sizes.off_norms, 0, ctx->total_mats * sizeof(float));
  if (ce == cudaSuccess) ce = cudaMemset(ctx->ws + ctx->sizes.off_rms, 0, ctx->total_mats * sizeof(float));
  if (ce == cudaSuccess) ce = cudaMemset(ctx->ws + ctx->sizes.off_debug, 0xFF, 1024 * sizeof(unsigned));
  if (ce != cudaSuccess) { delete ctx; return fail(MUON_ERR_CUDA, "workspace init: %s", cudaGetErrorString(ce)); }
  *out_ctx = ctx;
  return MUON_OK;
}

static int check_hparams(const muon_hparams* hp) {
  if (!hp) return fail(MUON_ERR_INVALID_ARG, "hparams is null");
  if (hp->ns_steps < 0 || hp->ns_steps > 64) return fail(MUON_ERR_INVALID_ARG, "ns_steps must be in [0, 64]");
  if (!(hp->eps >= 0.f)) return fail(MUON_ERR_INVALID_ARG, "eps must be >= 0");
  if (hp->scale_mode < MUON_SCALE_ADJUSTED_LR || hp->scale_mode > MUON_SCALE_UPDATE_NORM)
    return fail(MUON_ERR_INVALID_ARG, "unknown scale_mode");
  if (hp->scale_mode == MUON_SCALE_FIXED_DIM && !(hp->scale_dim > 0.f))
    return fail(MUON_ERR_INVALID_ARG, "scale_dim must be positive with MUON_SCALE_FIXED_DIM");
  for (int i = 0; hp->coeffs && i < 3 * hp->ns_steps; ++i)
    if (!std::isfinite(hp->coeffs[i])) return fail(MUON_ERR_INVALID_ARG, "coefficient schedule must be finite");
  if (!std::isfinite(hp->lr) || !std::isfinite(hp->wd) || !std::isfinite(hp->mu) || !std::isfinite(hp->a) ||
      !std::isfinite(hp->b) || !std::isfinite(hp->c) || !std::isfinite(hp->rms_scale))
    return fail(MUON_ERR_INVALID_ARG, "hyper-parameters must be finite");
  return MUON_OK;
}

// One Muon step for matrices [first, first + count) of bucket b (at most one
// chunk), enqueued on `stream`.
static int step_chunk(muon_ctx* ctx, const muon_hparams* hp, cudaStream_t stream, size_t b, int first, int count,
                      int* launch_counter) {
  int launches = 0;
  cudaError_t ce = cudaSuccess;
  DevStatus* status = reinterpret_cast<DevStatus*>(ctx->ws + ctx->sizes.off_status);
  float* norms = reinterpret_cast<float*>(ctx->ws + ctx->sizes.off_norms);
  Bucket& B = ctx->buckets[b];
  // factor of O in the update (Sec. 2.2 / Sec. 3.1): 0.2*sqrt(max(rows, cols)), or 0.2*sqrt(H)
  const float factor = hp->rms_scale * std::sqrt(hp->scale_mode == MUON_SCALE_FIXED_DIM
                                                     ? hp->scale_dim : static_cast<float>(B.n));
  const bool normalise = hp->scale_mode == MUON_SCALE_UPDATE_NORM;
  // The last epilogue updates W when every W of the bucket is TMA-addressable
  // (bf16 or fp32), the update needs no whole-matrix statistic, a*X is folded into the
  // product and the O tap is off; otherwise O is stored and a second pass applies it.
  const bool fused_update = B.fused_update && !normalise && B.fold_identity && !ctx->keep_o;
  const float upd_scale = -hp->lr * factor;
  const float decay = 1.0f - hp->lr * hp->wd;
  const MatDesc* descs = reinterpret_cast<const MatDesc*>(ctx->ws + B.off_descs) + first;
  MatScal* scal = reinterpret_cast<MatScal*>(ctx->ws + B.off_scal);
  float* partials = reinterpret_cast<float*>(ctx->ws + B.off_partials);

  const int stream_tiles = B.stream_tma ? B.stream_tiles_tma : B.stream_tiles_generic;
  const int* g_bad = nullptr;
  if (hp->protect_momentum) {
    // find the matrices with a non-finite gradient first, so that their momentum is left alone
    int* bad = reinterpret_cast<int*>(ctx->ws + B.off_bad);
    LaunchTimer lt(ctx, stream, MUON_KERNEL_NORM);
    ce = launch_grad_finite(descs, count, B.n, B.g_dtype == MUON_DTYPE_FP32, bad, stream);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "gradient check launch: %s", cudaGetErrorString(ce));
    ++launches;
    g_bad = bad;
  }
  if (B.stream_tma) {
    StreamTmaParams S{};
    S.map_x = B.x_b64[0];
    S.gmaps = reinterpret_cast<const CUtensorMap*>(ctx->ws + B.off_gmaps) + first;
    S.mmaps = reinterpret_cast<const CUtensorMap*>(ctx->ws + B.off_mmaps) + first;
    S.descs = descs;
    S.partials = partials;
    S.status = status;
    S.count = count;
    S.tiles_per_matrix = stream_tiles;
    S.m = B.m;
    S.n = B.n;
    S.mu = hp->mu;
    S.nesterov = hp->nesterov ? 1 : 0;
    S.g_bad = g_bad;
    LaunchTimer lt(ctx, stream, MUON_KERNEL_MOMENTUM);
    ce = launch_momentum_tma(S, B.g_dtype == MUON_DTYPE_FP32, ctx->num_sms, stream);
  } else {
    StreamParams S{};
    S.descs = descs;
    S.partials = partials;
    S.x = reinterpret_cast<__nv_bfloat16*>(ctx->ws + B.off_x[0]);
    S.x_stride = static_cast<long long>(B.x_stride);
    S.ldx = B.ldx;
    S.count = count;
    S.tiles_per_matrix = stream_tiles;
    S.mu = hp->mu;
    S.nesterov = hp->nesterov ? 1 : 0;
    S.g_bad = g_bad;
    LaunchTimer lt(ctx, stream, MUON_KERNEL_MOMENTUM);
    ce = launch_momentum_cast(S, B.g_dtype == MUON_DTYPE_FP32, stream);
  }
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "momentum kernel launch: %s", cudaGetErrorString(ce));
  ++launches;
  { LaunchTimer lt(ctx, stream, MUON_KERNEL_NORM); ce = launch_norm_finalise(partials, stream_tiles, count, hp->eps, descs, scal, norms, status, stream); }
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "norm kernel launch: %s", cudaGetErrorString(ce));
  ++launches;

  int cur = 0;
  int a_last = 0, b_last = 1;
  auto base_params = [&]() {
    GemmParams P{};
    P.descs = descs;
    P.scal = scal;
    P.status = status;
    P.debug = reinterpret_cast<unsigned*>(ctx->ws + ctx->sizes.off_debug);
    P.rms_partials = reinterpret_cast<float*>(ctx->ws + B.off_rms_partials);
    P.wmaps = reinterpret_cast<const CUtensorMap*>(ctx->ws + B.off_wmaps) + first;
    P.count = count;
    P.m = B.m;
    P.n_long = B.n;
    P.tiles_t = reinterpret_cast<const PairTile*>(ctx->ws + B.off_comb_tiles_t);
    P.upd_scale = upd_scale;
    P.decay = decay;
    return P;
  };
  // tile tables of the products with a symmetric result
  auto set_sym_tiles = [&](GemmParams& P) {
    P.tiles = reinterpret_cast<const PairTile*>(ctx->ws + B.off_sym_tiles);
    P.tiles_tail = reinterpret_cast<const PairTile*>(ctx->ws + B.off_sym_tiles_tail);
    P.tiles_per_unit = static_cast<int>(B.sym_tiles.size());
    P.tiles_per_tail = static_cast<int>(B.sym_tiles_tail.size());
    P.unit_mats = B.sym_unit_mats;
  };
  // S[out] = X X^T (first iteration: times s^2, the deferred normalisation)
  auto gram = [&](int x, int out, bool first_it) {
    GemmParams P = base_params();
    P.map_a = B.x_op[x];
    P.map_a64 = B.x_b64[x];  // unused
    P.map_b = B.x_b64[x];
    P.map_in = B.s_e[out];  // unused
    P.map_out = B.s_e[out];
    set_sym_tiles(P);
    P.k = B.n;
    P.out_cols = B.m;
    P.a_sym = 0; P.b_sym = 0; P.b_mn_major = 0;
    P.has_in = 0;
    P.scale_kind = first_it ? 1 : 0;
    P.last = 0;
    P.c_acc = 1.f; P.c_in = 0.f; P.diag_add = 0.f;
    LaunchTimer lt(ctx, stream, MUON_KERNEL_GRAM);
    ++launches;
    return launch_ns_gemm(P, B.sym_acc_cols, ctx->max_clusters, stream);
  };
  // S[out] = c_acc * S[left] S[right] + c_in * S[in] + diag * I for symmetric,
  // commuting operands kept as their upper blocks (in < 0: no input tile)
  auto sym_product = [&](int left, int right, int in, int out, float c_acc, float c_in, float diag) {
    GemmParams P = base_params();
    P.map_a = B.s_op[left];
    P.map_a64 = B.s_b64[left];
    P.map_b = B.s_b64[right];
    P.map_in = B.s_e[in < 0 ? out : in];
    P.map_out = B.s_e[out];
    set_sym_tiles(P);
    P.k = B.m;
    P.out_cols = B.m;
    P.a_sym = 1; P.b_sym = 1; P.b_mn_major = 0;
    P.has_in = in < 0 ? 0 : 1;
    P.scale_kind = 0;
    P.last = 0;
    P.c_acc = c_acc; P.c_in = in < 0 ? 0.f : c_in; P.diag_add = diag;
    LaunchTimer lt(ctx, stream, MUON_KERNEL_POLY);
    ++launches;
    return launch_ns_gemm(P, B.sym_acc_cols, ctx->max_clusters, stream);
  };
  // X[nxt] = co_a * X[cur] + S[s] X[cur] (co_a * X only when a*I is not folded into
  // S; first iteration: times s); the last iteration updates W in its epilogue
  // when every W of the bucket is TMA-addressable
  auto combine = [&](int s_buf, int x_cur, int x_nxt, bool first_it, bool fuse, float co_a) {
    GemmParams P = base_params();
    P.map_a = B.s_op[s_buf];
    P.map_a64 = B.s_b64[s_buf];
    P.map_b = B.x_b64[x_cur];
    P.map_in = B.x_e[x_cur];
    P.map_out = B.x_e[x_nxt];
    P.tiles = reinterpret_cast<const PairTile*>(ctx->ws + B.off_comb_tiles);
    P.tiles_tail = P.tiles;
    P.tiles_per_unit = static_cast<int>(B.comb_tiles.size());
    P.tiles_per_tail = 0;
    P.unit_mats = 1;
    P.k = B.m;
    P.out_cols = B.n;
    P.a_sym = 1; P.b_sym = 0; P.b_mn_major = 1;
    P.has_in = (fuse || !B.fold_identity) ? 1 : 0;  // W when fused, else X for the a*X term
    P.scale_kind = first_it ? 2 : 0;
    P.last = fuse ? 1 : 0;
    P.w_fp32 = B.w_dtype == MUON_DTYPE_FP32 ? 1 : 0;
    P.c_acc = 1.f; P.c_in = B.fold_identity ? 0.f : co_a;
    P.diag_add = 0.f;
    LaunchTimer lt(ctx, stream, MUON_KERNEL_COMB);
    ++launches;
    return launch_ns_gemm(P, B.comb_acc_cols, ctx->max_clusters, stream);
  };
  auto coef = [&](int it, int which) {
    return hp->coeffs ? hp->coeffs[3 * it + which] : (which == 0 ? hp->a : (which == 1 ? hp->b : hp->c));
  };
  // the mode the plan was made with, whatever the knob says now
  int pairs_left = B.pair_fold ? plan_pairs(B.pair_mode, B.m, B.n, B.fold_identity, hp->ns_steps) : 0;
  for (int it = 0; it < hp->ns_steps;) {
    const bool first_it = (it == 0);
    const bool pair = pairs_left > 0 && it + 1 < hp->ns_steps;
    if (pair) --pairs_left;
    const bool last_it = it + (pair ? 2 : 1) == hp->ns_steps;
    const int nxt = cur ^ 1;
    const float fold_a = B.fold_identity ? coef(it, 0) : 0.f;
    // A = X X^T;  B' = b*A + c*A*A (+ a*I)
    ce = gram(cur, 0, first_it);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "gram kernel launch: %s", cudaGetErrorString(ce));
    ce = sym_product(0, 0, 0, 1, coef(it, 2), coef(it, 1), fold_a);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "poly kernel launch: %s", cudaGetErrorString(ce));
    int s_comb = 1;
    a_last = 0;
    b_last = 1;
    if (pair) {
      // the next iteration without X: A' = B'^2 A, B'' = b'*A' + c'*A'^2 + a'*I, then B'' B'
      // (a product of two different matrices leaves diagonal blocks whose triangles
      // differ by rounding: they are made equal before anything reads them)
      auto symmetrise = [&](int buf) {
        LaunchTimer lt(ctx, stream, MUON_KERNEL_NORM);  // counted with the small helper kernels
        ++launches;
        return launch_symmetrise_diag(reinterpret_cast<__nv_bfloat16*>(ctx->ws + B.off_s[buf]),
                                      static_cast<long long>(B.a_stride), B.lda, B.m, count, stream);
      };
      ce = sym_product(1, 1, -1, 2, 1.f, 0.f, 0.f);
      if (ce == cudaSuccess) ce = sym_product(2, 0, -1, 3, 1.f, 0.f, 0.f);
      if (ce == cudaSuccess) ce = symmetrise(3);
      if (ce == cudaSuccess) ce = sym_product(3, 3, 3, 2, coef(it + 1, 2), coef(it + 1, 1), coef(it + 1, 0));
      if (ce == cudaSuccess) ce = sym_product(2, 1, -1, 0, 1.f, 0.f, 0.f);
      // B'' B' only multiplies X; in the first pair its mismatch stays at rounding level
      // (no polynomial is formed from it), later pairs are near the band and keep the fix
      if (ce == cudaSuccess && !first_it) ce = symmetrise(0);
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "poly kernel launch: %s", cudaGetErrorString(ce));
      s_comb = 0;
      a_last = 3;
      b_last = 2;
    }
    ce = combine(s_comb, cur, nxt, first_it, last_it && fused_update, coef(it, 0));
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "combine kernel launch: %s", cudaGetErrorString(ce));
    cur = nxt;
    it += pair ? 2 : 1;
  }
  {
    // Update RMS for logging (Algorithm 1, returned value) and, when the
    // weights were not updated in the last epilogue (no iteration, fp32 or
    // TMA-unaddressable weights, normalised update), the separate update
    // W <- decay*W - lr*f*O from the stored O.
    float* rms = reinterpret_cast<float*>(ctx->ws + ctx->sizes.off_rms);
    float* rms_partials = reinterpret_cast<float*>(ctx->ws + B.off_rms_partials);
    const int per_matrix = static_cast<int>(B.comb_tiles.size()) * 8;
    if (hp->ns_steps > 0 && fused_update) {
      LaunchTimer lt(ctx, stream, MUON_KERNEL_NORM);
      ce = launch_rms_finalise(rms_partials, per_matrix, count, factor, descs, scal, false, hp->rms_scale, false, rms,
                               nullptr, stream);
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "rms kernel launch: %s", cudaGetErrorString(ce));
      ++launches;
    } else {
      float* factors = reinterpret_cast<float*>(ctx->ws + B.off_factors);
      const __nv_bfloat16* xo = reinterpret_cast<const __nv_bfloat16*>(ctx->ws + B.off_x[cur]);
      {
        LaunchTimer lt(ctx, stream, MUON_KERNEL_NORM);
        ce = launch_sumsq_x(xo, static_cast<long long>(B.x_stride), B.ldx, B.m, B.n, count, per_matrix, rms_partials,
                            stream);
        if (ce == cudaSuccess)
          ce = launch_rms_finalise(rms_partials, per_matrix, count, factor, descs, scal, hp->ns_steps == 0,
                                   hp->rms_scale, normalise, rms, factors, stream);
      }
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "rms kernel launch: %s", cudaGetErrorString(ce));
      launches += 2;
      {
        LaunchTimer lt(ctx, stream, MUON_KERNEL_UPDATE);
        ce = launch_update_from_x(descs, scal, factors, xo, static_cast<long long>(B.x_stride), B.ldx, count,
                                  B.m, B.n, -hp->lr, decay, B.w_dtype == MUON_DTYPE_FP32, stream);
      }
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "update kernel launch: %s", cudaGetErrorString(ce));
      ++launches;
    }
  }
  ctx->x0_buf[b] = 0;
  ctx->xlast_buf[b] = cur;
  ctx->a_last_buf[b] = a_last;
  ctx->b_last_buf[b] = b_last;
  *launch_counter += launches;
  return MUON_OK;
}

int muon_step(muon_ctx* ctx, const muon_hparams* hp, void* stream_v) {
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "ctx is null");
  DeviceGuard guard(ctx->device);
  int rc = check_hparams(hp);
  if (rc) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  int launches = 0;
  for (size_t b = 0; b < ctx->buckets.size(); ++b) {
    const Bucket& B = ctx->buckets[b];
    const int total = static_cast<int>(B.mats.size());
    for (int first = 0; first < total; first += B.chunk) {
      rc = step_chunk(ctx, hp, stream, b, first, std::min(B.chunk, total - first), &launches);
      if (rc) return rc;
    }
  }
  ctx->last_launches = launches;
  return MUON_OK;
}

int muon_step_bucket(muon_ctx* ctx, const muon_hparams* hp, int bucket, void* stream_v) {
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "ctx is null");
  if (bucket < 0 || bucket >= static_cast<int>(ctx->buckets.size()))
    return fail(MUON_ERR_INVALID_ARG, "bucket %d out of range (context has %zu)", bucket, ctx->buckets.size());
  DeviceGuard guard(ctx->device);
  int rc = check_hparams(hp);
  if (rc) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  int launches = 0;
  const Bucket& B = ctx->buckets[bucket];
  const int total = static_cast<int>(B.mats.size());
  for (int first = 0; first < total; first += B.chunk) {
    rc = step_chunk(ctx, hp, stream, bucket, first, std::min(B.chunk, total - first), &launches);
    if (rc) return rc;
  }
  ctx->last_launches = launches;
  return MUON_OK;
}

int muon_step_host(muon_ctx* ctx, const muon_hparams* hp, const void* const* const* g_host,
                   void* const* const* w_host, void* stream_v) {
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "ctx is null");
  DeviceGuard guard(ctx->device);
  if (!g_host) return fail(MUON_ERR_INVALID_ARG, "g_host is null");
  int rc = check_hparams(hp);
  if (rc) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  cudaError_t ce = cudaSuccess;
  if (!ctx->s_in) {
    ce = cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking);
    if (ce == cudaSuccess) ce = cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "copy stream creation: %s", cudaGetErrorString(ce));
  }
  size_t ev_next = 0;
  auto next_event = [&](cudaEvent_t* out) -> cudaError_t {
    if (ev_next == ctx->pipe_events.size()) {
      cudaEvent_t e;
      cudaError_t r = cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
      if (r != cudaSuccess) return r;
      ctx->pipe_events.push_back(e);
    }
    *out = ctx->pipe_events[ev_next++];
    return cudaSuccess;
  };
  // Uploads, kernels and downloads of successive slices of a bucket overlap:
  // slice k+1 is uploaded on one copy stream while slice k runs on the caller's
  // stream and slice k-1 is downloaded on the other copy stream.
  cudaEvent_t ev;
  ce = next_event(&ev);
  if (ce == cudaSuccess) ce = cudaEventRecord(ev, stream);             // copies start after earlier work
  if (ce == cudaSuccess) ce = cudaStreamWaitEvent(ctx->s_in, ev, 0);
  if (ce == cudaSuccess) ce = cudaStreamWaitEvent(ctx->s_out, ev, 0);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "stream ordering: %s", cudaGetErrorString(ce));
  int launches = 0;
  for (size_t b = 0; b < ctx->buckets.size(); ++b) {
    const Bucket& B = ctx->buckets[b];
    const int total = static_cast<int>(B.mats.size());
    // Slices of about kHostSliceBytes of gradients: short enough that the first upload and the last
    // download, which nothing overlaps, are a small part of the step, long enough to keep the launches few.
    const size_t g_bytes_per_mat = static_cast<size_t>(B.m) * B.n * (B.g_dtype == MUON_DTYPE_FP32 ? 4 : 2);
    const int slice = static_cast<int>(std::max<size_t>(1, std::min<size_t>(B.chunk, std::max<size_t>(1, kHostSliceBytes / g_bytes_per_mat))));
    for (int first = 0; first < total; first += slice) {
      const int count = std::min(slice, total - first);
      for (int i = first; i < first + count && ce == cudaSuccess; ++i) {
        const MatRef& r = B.mats[i];
        const muon_group& G = ctx->groups[r.group];
        const size_t es = G.g_dtype == MUON_DTYPE_FP32 ? 4 : 2;
        if (G.ld_g == G.cols)  // dense on both sides: one linear copy
          ce = cudaMemcpyAsync(const_cast<void*>(G.g[r.index]), g_host[r.group][r.index],
                               static_cast<size_t>(G.rows) * G.cols * es, cudaMemcpyHostToDevice, ctx->s_in);
        else
          ce = cudaMemcpy2DAsync(const_cast<void*>(G.g[r.index]), G.ld_g * es, g_host[r.group][r.index], G.cols * es,
                                 G.cols * es, G.rows, cudaMemcpyHostToDevice, ctx->s_in);
      }
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "gradient upload: %s", cudaGetErrorString(ce));
      ce = next_event(&ev);
      if (ce == cudaSuccess) ce = cudaEventRecord(ev, ctx->s_in);
      if (ce == cudaSuccess) ce = cudaStreamWaitEvent(stream, ev, 0);
      if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "stream ordering: %s", cudaGetErrorString(ce));
      rc = step_chunk(ctx, hp, stream, b, first, count, &launches);
      if (rc) return rc;
      if (w_host) {
        ce = next_event(&ev);
        if (ce == cudaSuccess) ce = cudaEventRecord(ev, stream);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(ctx->s_out, ev, 0);
        for (int i = first; i < first + count && ce == cudaSuccess; ++i) {
          const MatRef& r = B.mats[i];
          const muon_group& G = ctx->groups[r.group];
          const size_t es = G.w_dtype == MUON_DTYPE_FP32 ? 4 : 2;
          if (G.ld_w == G.cols)
            ce = cudaMemcpyAsync(w_host[r.group][r.index], G.w[r.index], static_cast<size_t>(G.rows) * G.cols * es,
                                 cudaMemcpyDeviceToHost, ctx->s_out);
          else
            ce = cudaMemcpy2DAsync(w_host[r.group][r.index], G.cols * es, G.w[r.index], G.ld_w * es, G.cols * es,
                                   G.rows, cudaMemcpyDeviceToHost, ctx->s_out);
        }
        if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "weight download: %s", cudaGetErrorString(ce));
      }
    }
  }
  // the caller's stream completes only when the last download has
  ce = next_event(&ev);
  if (ce == cudaSuccess) ce = cudaEventRecord(ev, ctx->s_out);
  if (ce == cudaSuccess) ce = cudaStreamWaitEvent(stream, ev, 0);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "stream ordering: %s", cudaGetErrorString(ce));
  ctx->last_launches = launches;
  return MUON_OK;
}

int muon_status(muon_ctx* ctx, void* stream_v, int* device_status, int* matrix_index) {
  if (!ctx || !device_status) return fail(MUON_ERR_INVALID_ARG, "ctx or device_status is null");
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  DevStatus st{0, -1};
  cudaError_t ce = cudaMemcpyAsync(&st, ctx->ws + ctx->sizes.off_status, sizeof(st), cudaMemcpyDeviceToHost, stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "status read: %s", cudaGetErrorString(ce));
  *device_status = st.code;
  if (matrix_index) *matrix_index = st.code ? st.matrix : -1;
  if (st.code) {
    DevStatus init{0, -1};
    ce = cudaMemcpyAsync(ctx->ws + ctx->sizes.off_status, &init, sizeof(init), cudaMemcpyHostToDevice, stream);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "status clear: %s", cudaGetErrorString(ce));
  }
  return MUON_OK;
}

int muon_get_norms(muon_ctx* ctx, void* stream_v, float* out, int n) {
  if (!ctx || !out || n < 0 || n > ctx->total_mats) return fail(MUON_ERR_INVALID_ARG, "bad arguments");
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  cudaError_t ce = cudaMemcpyAsync(out, ctx->ws + ctx->sizes.off_norms, n * sizeof(float), cudaMemcpyDeviceToHost, stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "norm read: %s", cudaGetErrorString(ce));
  return MUON_OK;
}

int muon_get_update_rms(muon_ctx* ctx, void* stream_v, float* out, int n) {
  if (!ctx || !out || n < 0 || n > ctx->total_mats) return fail(MUON_ERR_INVALID_ARG, "bad arguments");
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  cudaError_t ce = cudaMemcpyAsync(out, ctx->ws + ctx->sizes.off_rms, n * sizeof(float), cudaMemcpyDeviceToHost, stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "rms read: %s", cudaGetErrorString(ce));
  return MUON_OK;
}

int muon_destroy(muon_ctx* ctx) {
  delete ctx;
  return MUON_OK;
}

int muon_last_launch_count(const muon_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

int muon_profile_enable(muon_ctx* ctx, int enable) {
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "ctx is null");
  ctx->profile = enable ? 1 : 0;
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  return MUON_OK;
}

int muon_profile_read(muon_ctx* ctx, double* ms_by_kernel, int* launches_by_kernel) {
  if (!ctx || !ms_by_kernel || !launches_by_kernel) return fail(MUON_ERR_INVALID_ARG, "null argument");
  DeviceGuard guard(ctx->device);
  for (int k = 0; k < MUON_KERNEL_KINDS; ++k) { ms_by_kernel[k] = 0.0; launches_by_kernel[k] = 0; }
  cudaError_t ce = cudaDeviceSynchronize();
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "synchronise: %s", cudaGetErrorString(ce));
  for (size_t i = 0; i * 2 + 1 < ctx->ev_used + 1 && i < ctx->ev_kind.size(); ++i) {
    float ms = 0.f;
    ce = cudaEventElapsedTime(&ms, ctx->ev_pool[2 * i], ctx->ev_pool[2 * i + 1]);
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "event elapsed: %s", cudaGetErrorString(ce));
    ms_by_kernel[ctx->ev_kind[i]] += ms;
    launches_by_kernel[ctx->ev_kind[i]] += 1;
  }
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  return MUON_OK;
}

int muon_debug_tmem_bases(muon_ctx* ctx, unsigned* out_host, int n) {
  if (!ctx || !out_host || n < 0 || n > 1024) return fail(MUON_ERR_INVALID_ARG, "bad arguments");
  DeviceGuard guard(ctx->device);
  cudaError_t ce = cudaDeviceSynchronize();
  if (ce == cudaSuccess)
    ce = cudaMemcpy(out_host, ctx->ws + ctx->sizes.off_debug, n * sizeof(unsigned), cudaMemcpyDeviceToHost);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "debug read: %s", cudaGetErrorString(ce));
  return MUON_OK;
}

int muon_debug_wait_expiry(muon_ctx* ctx, void* stream_v, int matrix_index, unsigned limit_ms) {
  if (!ctx || matrix_index < 0 || matrix_index >= ctx->total_mats || limit_ms == 0 || limit_ms > 1000)
    return fail(MUON_ERR_INVALID_ARG, "bad arguments (limit_ms must be 1..1000)");
  DeviceGuard guard(ctx->device);
  DevStatus* status = reinterpret_cast<DevStatus*>(ctx->ws + ctx->sizes.off_status);
  cudaError_t ce = launch_wait_expiry_probe(status, matrix_index, static_cast<unsigned long long>(limit_ms) * 1000000ull,
                                            static_cast<cudaStream_t>(stream_v));
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "probe launch: %s", cudaGetErrorString(ce));
  return MUON_OK;
}

int muon_debug_keep(muon_ctx* ctx, int keep) {
  if (!ctx) return fail(MUON_ERR_INVALID_ARG, "ctx is null");
  ctx->keep_o = keep ? 1 : 0;
  return MUON_OK;
}

int muon_debug_read(muon_ctx* ctx, int matrix_index, int which, void* dst_host, size_t dst_bytes) {
  if (!ctx || !dst_host) return fail(MUON_ERR_INVALID_ARG, "ctx or dst is null");
  if (matrix_index < 0 || matrix_index >= ctx->total_mats) return fail(MUON_ERR_INVALID_ARG, "matrix index out of range");
  DeviceGuard guard(ctx->device);
  const int b = ctx->where[matrix_index].first, pos = ctx->where[matrix_index].second;
  const Bucket& B = ctx->buckets[b];
  if (ctx->buckets.size() != 1 || static_cast<int>(B.mats.size()) > B.chunk)
    return fail(MUON_ERR_UNSUPPORTED, "taps need a context with one shape bucket that fits one chunk");
  const uint8_t* src;
  int rows, cols, ld;
  switch (which) {
    case MUON_TAP_X0:
      src = ctx->ws + B.off_x[ctx->x0_buf[b]] + static_cast<size_t>(pos) * B.x_stride * 2;
      rows = B.m; cols = B.n; ld = B.ldx;
      break;
    case MUON_TAP_X:
      src = ctx->ws + B.off_x[ctx->xlast_buf[b]] + static_cast<size_t>(pos) * B.x_stride * 2;
      rows = B.m; cols = B.n; ld = B.ldx;
      break;
    case MUON_TAP_A:
      src = ctx->ws + B.off_s[ctx->a_last_buf[b]] + static_cast<size_t>(pos) * B.a_stride * 2;
      rows = B.m; cols = B.m; ld = B.lda;
      break;
    case MUON_TAP_B:
      src = ctx->ws + B.off_s[ctx->b_last_buf[b]] + static_cast<size_t>(pos) * B.a_stride * 2;
      rows = B.m; cols = B.m; ld = B.lda;
      break;
    default:
      return fail(MUON_ERR_INVALID_ARG, "unknown tap");
  }
  if (dst_bytes < static_cast<size_t>(rows) * cols * 2) return fail(MUON_ERR_INVALID_ARG, "destination too small");
  cudaError_t ce = cudaDeviceSynchronize();
  if (ce == cudaSuccess)
    ce = cudaMemcpy2D(dst_host, static_cast<size_t>(cols) * 2, src, static_cast<size_t>(ld) * 2,
                      static_cast<size_t>(cols) * 2, rows, cudaMemcpyDeviceToHost);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "tap read: %s", cudaGetErrorString(ce));
  if (which == MUON_TAP_A || which == MUON_TAP_B) {
    // the kernels keep only the 128-blocks on or above the diagonal: fill the rest by symmetry
    uint16_t* d = static_cast<uint16_t*>(dst_host);
    for (int i = 0; i < rows; ++i)
      for (int j = 0; j < (i / 128) * 128; ++j) d[static_cast<size_t>(i) * cols + j] = d[static_cast<size_t>(j) * cols + i];
  }
  return MUON_OK;
}

}  // extern "C"
