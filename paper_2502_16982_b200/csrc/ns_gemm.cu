// Newton-Schulz GEMM kernel for sm_100a (Eq. 2 of the paper, factored as
//   A = X X^T,   B = b*A + c*A*A,   X' = a*X + B X).
// One persistent, warp-specialised kernel on CTA pairs serves all three products.
//
// Two CTAs on neighbouring SMs form a cluster and share one UMMA
// (tcgen05.mma.cta_group::2): M = 256 (128 rows from each CTA's own A tile),
// N = 128 or 256 with the B operand split between the two CTAs' shared
// memories, so each CTA stages only half of B.  Which rows and columns a tile
// covers comes from a table built on the host (PairTile): the two CTAs' row
// blocks, even their matrices, need not be the same.
//
// Per CTA (192 threads):
//   warp 0      TMA producer: its 128x64 A tile and its half of the B tile per
//               K block into a kStages-deep ring; byte counts of both CTAs are
//               reported to the leader CTA's "full" barrier.  No multicast.
//   warp 1      leader CTA only: UMMA issuer; tcgen05.commit (to both CTAs'
//               barriers) frees ring slots and publishes accumulators (two
//               TMEM stages of up to 256 fp32 columns).
//   warps 2-5   epilogue.  Each warp owns the 32 accumulator rows its TMEM lane
//               quarter holds and runs its own pipeline over "quarters" (32
//               rows x 64 columns): quarter g uses ring entry g % R of the
//               warp's staging.  An entry is filled by TMA with the epilogue's
//               input tile (A for the polynomial, X for the combine, W and X on
//               the last iteration) R-1 quarters ahead, combined in place with
//               the accumulator (tcgen05.ld, fp32 arithmetic, one bf16
//               rounding) and written back by a TMA store issued by the warp
//               itself; the warps never wait for one another.
//
// A tile may also be half height (M = 128: 64 rows per CTA, both halves of one
// row block).  The accumulator then lies differently in TMEM: lanes 0-63 of a
// CTA hold its 64 rows against the first half of the N columns, lanes 64-127 the
// same rows against the second half (both in TMEM columns [0, N/2)), so epilogue
// warp q owns rows 32 (q & 1) .. + 31 of the CTA and column half q >> 1.
//
// Symmetric matrices (A and B) are kept as their 128x128 blocks on or above
// the diagonal only.  The products that produce them follow a tile table that
// covers exactly those blocks (a table entry says which blocks of a tile are
// stored: a block under the diagonal, or the cross blocks of a tile shared by
// two matrices, are computed and dropped); the products that consume them read
// a block below the diagonal as the transpose of its mirror image (an MN-major
// UMMA operand), so both triangles are the same bits by construction.
//
// The combine is a*X + B X.  For buckets whose short side is at least 16 the
// polynomial's epilogue adds a to the diagonal of B in fp32 before the one bf16
// rounding (B' = B + a*I), so that the combine is the single product B' X and
// its epilogue loads no X tile; smaller matrices keep the a*X term in the
// combine's epilogue (for them the rounding of B_ii + a is the larger error).
//
// Last iteration (Sec. 2.2): the entry holds the W tile,
//   O = scale * acc,   W <- (1 - lr*wd) * W - lr * rms_scale * sqrt(max(rows, cols)) * O
// in fp32; O itself never reaches HBM.  (W is bf16, or fp32 in the kWFp32
// instantiation, where an entry is two boxes of 32 fp32 columns and an optional
// bf16 copy of the new weights is written from the registers.)  For a matrix stored with rows > cols
// (Newton-Schulz ran on its transpose) the last product is formed transposed,
// O^T = X^T B' with X^T read as an MN-major operand from X and the symmetric B'
// as the other operand, so that the tile comes out in W's own orientation and
// no transposition is needed; such tiles follow a second tile table (row pairs
// along the long side).
//
// Every software wait is bounded (ptx::mbar_wait); on expiry the CTA records
// MUON_ERR_TIMEOUT, all roles drain, both CTAs meet at the final cluster
// barrier, TMEM is freed and the kernel returns.
#include <cuda_bf16.h>

#include <type_traits>

#include "internal.h"
#include "ptx.cuh"

namespace muon {

namespace {

// Shared memory is split between the operand ring and the epilogue staging.
// A product whose epilogue loads no input tile (the Gram product) does best
// with a deeper ring (5 stages, 4 staging buffers per warp); the others with 4
// stages and 6 buffers (measured on the expert bucket).
constexpr int kMaxStages = 5;
constexpr int kMaxSubs = 6;
constexpr int kTileABytes = 128 * kBK * 2;   // 16 KiB: this CTA's 128 A rows
constexpr int kTileBBytes = 128 * kBK * 2;   // 16 KiB: up to 128 B rows (half of N = 256)
constexpr int kStageBytes = kTileABytes + kTileBBytes;
constexpr int kEpiWarps = 4;
constexpr int kSubBytes = 32 * 128;          // one warp's 32 rows x 64 bf16 columns
constexpr int kNumAcc = 2;

struct Barriers {
  unsigned long long full[kMaxStages];    // leader's copy is the live one
  unsigned long long empty[kMaxStages];
  unsigned long long acc_full[kNumAcc];
  unsigned long long acc_empty[kNumAcc];  // leader's copy is the live one
  unsigned long long io_ready[kEpiWarps][kMaxSubs];  // ring entry filled / free to write
  uint32_t tmem_base;
  int abort_flag;
};

constexpr int kBarrierBytes = 512;
constexpr int kSubBytesFp32 = 2 * kSubBytes;  // the same quarter of an fp32 W: two boxes of 32 columns
constexpr int smem_bytes(int stages, int subs, int entry_bytes = kSubBytes) {
  return 1024 + stages * kStageBytes + kEpiWarps * subs * entry_bytes + kBarrierBytes;
}
static_assert(sizeof(Barriers) <= kBarrierBytes, "barrier block too large");
static_assert(smem_bytes(5, 4) <= 232448 && smem_bytes(4, 6) <= 232448 && smem_bytes(4, 3, kSubBytesFp32) <= 232448,
              "exceeds the 227 KiB shared-memory limit");
static_assert(kBK == 64, "the issuer loop issues four K = 16 steps per stage");

__device__ __forceinline__ void report_timeout(const GemmParams& P, int mat) {
  if (atomicCAS(&P.status->code, 0, -6 /* MUON_ERR_TIMEOUT */) == 0) {
    P.status->matrix = P.descs[mat].global_index;
  }
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ void unpack8(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, float (&f)[8]) {
  f[0] = __uint_as_float(w0 << 16); f[1] = __uint_as_float(w0 & 0xFFFF0000u);
  f[2] = __uint_as_float(w1 << 16); f[3] = __uint_as_float(w1 & 0xFFFF0000u);
  f[4] = __uint_as_float(w2 << 16); f[5] = __uint_as_float(w2 & 0xFFFF0000u);
  f[6] = __uint_as_float(w3 << 16); f[7] = __uint_as_float(w3 & 0xFFFF0000u);
}

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t& w0, uint32_t& w1, uint32_t& w2, uint32_t& w3) {
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(addr));
}

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
}

// What one tile of the launch computes: its table entry, the first matrix of
// its unit, whether it is a transposed-formulation tile of the last iteration,
// and up to which K block each operand is read transposed (MN-major).
struct TilePlan {
  PairTile pt;
  int base_mat;
  bool swapped;
  int kb_a, kb_b;  // K blocks [0, kb_a) of A and [0, kb_b) of B are read MN-major
};

// Field of CTA `rank` of a table entry, without indexing an array at run time
// (which would put the entry in local memory).
template <typename T>
__device__ __forceinline__ int of_rank(const T (&v)[2], int rank) {
  return rank ? static_cast<int>(v[1]) : static_cast<int>(v[0]);
}

// Table entry and first matrix of tile `tile` of the launch: whole units first,
// then the tiles of a last matrix that has no partner.
__device__ __forceinline__ void locate_tile(const GemmParams& P, int tile, PairTile& pt, int& base_mat, bool& swapped) {
  const int unit = tile / P.tiles_per_unit;
  const int full_units = P.count / P.unit_mats;
  swapped = false;
  if (unit < full_units) {
    base_mat = unit * P.unit_mats;
    const int idx = tile - unit * P.tiles_per_unit;
    swapped = P.last && P.descs[base_mat].transposed != 0;  // the last product has one matrix per unit
    pt = (swapped ? P.tiles_t : P.tiles)[idx];
  } else {
    base_mat = full_units * P.unit_mats;
    pt = P.tiles_tail[tile - full_units * P.tiles_per_unit];
  }
}

__device__ __forceinline__ TilePlan plan_tile(const GemmParams& P, int tile, int num_kb) {
  TilePlan t;
  locate_tile(P, tile, t.pt, t.base_mat, t.swapped);
  // A symmetric operand kept as its upper blocks is read transposed up to the
  // K block where a row of the operand tile is still below the diagonal.  One
  // instruction reads the tiles of both CTAs in one layout, so their blocks
  // are equal or neighbours and the later switch point serves both: the block
  // the other CTA then reads "the wrong way round" is a diagonal block, which
  // is the same bits either way.
  const int sym_a = min(num_kb, 2 * max(t.pt.i[0], t.pt.i[1]));
  const int sym_b = min(num_kb, 2 * (t.pt.nbw == 2 ? max(t.pt.j[0], t.pt.j[1]) : t.pt.j[0]));
  if (t.swapped) {  // A = X^T from X (MN-major throughout), B = the symmetric matrix
    t.kb_a = num_kb;
    t.kb_b = sym_b;
  } else {
    t.kb_a = P.a_sym ? sym_a : 0;
    t.kb_b = P.b_mn_major ? num_kb : (P.b_sym ? sym_b : 0);
  }
  return t;
}

// Walks the stream of 64-column quarters one epilogue warp processes: tiles in
// the CTA pair's order, within a tile the quarters that hold output of this warp
// (`qmask`: bit s set = the 32 rows x 64 columns at TMEM columns [64 s, 64 s + 64)
// of the warp's lanes are still to be stored).
struct QuarterCursor {
  int tile, mat;
  unsigned qmask;
  int ib;         // row block of the output
  int row0;       // first of this warp's 32 output rows
  int cb0, cb1;   // column block of quarters {0, 1} and of quarters {2, 3}
  int cofs;       // column offset inside the block on top of 64 (s & 1)
  int row_limit;  // output rows of the matrix in this tile's orientation

  // Quarters of tile `t` for warp `q` of CTA `rank`; returns false past the last tile.
  __device__ __forceinline__ bool open_tile(const GemmParams& P, int t, int total_tiles, int rank, int q) {
    tile = t;
    if (t >= total_tiles) {
      qmask = 0;
      return false;
    }
    PairTile pt;
    int base_mat;
    bool swapped;
    locate_tile(P, t, pt, base_mat, swapped);
    row_limit = swapped ? P.n_long : P.m;
    const int col_limit = swapped ? P.m : P.out_cols;
    unsigned keep, slots;
    if (pt.half) {
      // half height: lanes 0-63 of the CTA (warps 0, 1) hold its 64 rows against the first half of the
      // N columns, lanes 64-127 (warps 2, 3) against the second half, both in TMEM columns [0, N/2)
      const int ch = q >> 1;
      mat = base_mat + pt.dm[0];
      ib = pt.i[0];
      row0 = ib * 128 + rank * 64 + (q & 1) * 32;
      if (pt.nbw == 2) {
        cb0 = cb1 = ch ? pt.j[1] : pt.j[0];
        cofs = 0;
        slots = 3u;
        keep = ((static_cast<unsigned>(pt.keep[0]) >> ch) & 1u) ? 3u : 0u;
      } else {
        cb0 = cb1 = pt.j[0];
        cofs = ch * 64;
        slots = 1u;
        keep = (pt.keep[0] & 1u) ? 1u : 0u;
      }
    } else {
      mat = base_mat + of_rank(pt.dm, rank);
      ib = of_rank(pt.i, rank);
      row0 = ib * 128 + q * 32;
      cb0 = pt.j[0];
      cb1 = pt.j[1];
      cofs = 0;
      slots = pt.nbw == 2 ? 15u : 3u;
      const unsigned k2 = static_cast<unsigned>(of_rank(pt.keep, rank));
      keep = ((k2 & 1u) ? 3u : 0u) | ((k2 & 2u) ? 12u : 0u);
    }
    qmask = 0;
    if (ib * 128 < row_limit) {  // else a ragged pair: nothing of ours
#pragma unroll
      for (int sl = 0; sl < 4; ++sl) {
        const bool on = ((slots & keep) >> sl & 1u) && col0(sl) < col_limit;
        qmask |= on ? (1u << sl) : 0u;
      }
    }
    return true;
  }
  __device__ __forceinline__ bool has_quarter() const { return qmask != 0; }
  __device__ __forceinline__ int quarter() const { return __ffs(qmask) - 1; }
  __device__ __forceinline__ void pop_quarter() { qmask &= qmask - 1; }
  __device__ __forceinline__ int col_block(int sl) const { return (sl >> 1) ? cb1 : cb0; }
  // offset of quarter sl's first column inside its column block, and that column itself
  __device__ __forceinline__ int col_in_block(int sl) const { return (sl & 1) * 64 + cofs; }
  __device__ __forceinline__ int col0(int sl) const { return col_block(sl) * 128 + col_in_block(sl); }
};

// kAccCols: fp32 TMEM columns per accumulator stage = widest N (128 or 256).
// kStages: depth of the operand ring; kSubsPerWarp: staging buffers per epilogue warp.
// kWFp32: the launch is a last iteration over fp32 weights (a staging buffer then
// holds 32 rows x 64 fp32 columns as two 128-byte-swizzled boxes of 32 columns).
template <int kAccCols, int kStages, int kSubsPerWarp, bool kWFp32 = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
ns_gemm_kernel(const __grid_constant__ GemmParams P) {
  constexpr int kEntryBytes = kWFp32 ? kSubBytesFp32 : kSubBytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* s_epi = smem + kStages * kStageBytes;
  Barriers* bars = reinterpret_cast<Barriers*>(s_epi + kEpiWarps * kSubsPerWarp * kEntryBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();      // 0 = leader
  const int cluster = static_cast<int>(ptx::cluster_id_x());
  const int num_clusters = static_cast<int>(ptx::num_clusters_x());
  const int total_tiles = (P.count / P.unit_mats) * P.tiles_per_unit + (P.count % P.unit_mats ? P.tiles_per_tail : 0);
  const int num_kb = (P.k + kBK - 1) / kBK;
  volatile int* abort_flag = &bars->abort_flag;
  constexpr uint32_t kTmemCols = kNumAcc * kAccCols;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
    }
    for (int s = 0; s < kNumAcc; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[s]), 2 * kEpiWarps);
    }
    for (int w = 0; w < kEpiWarps; ++w)
      for (int s = 0; s < kSubsPerWarp; ++s) ptx::mbar_init(ptx::smem_u32(&bars->io_ready[w][s]), 1);
    bars->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&P.map_a);
    ptx::prefetch_tensormap(&P.map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&bars->tmem_base), kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();  // both CTAs' barriers are initialised, both TMEM allocations done
  ptx::tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  // Everything above touched only this CTA's shared memory, TMEM and the kernel's parameters, so
  // it may overlap the tail of the previous kernel of the stream; its results are needed from here on.
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  if (P.debug != nullptr && threadIdx.x == 0) P.debug[blockIdx.x] = tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------ TMA producer ----
    // The whole warp walks the loop (so that its counters stay warp-uniform);
    // one elected lane issues the copies.
    {
      const bool elected = ptx::elect_one();
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      const uint32_t ring_u32 = ptx::smem_u32(ring);
      const uint32_t full0 = ptx::smem_u32(&bars->full[0]);
      const uint32_t empty0 = ptx::smem_u32(&bars->empty[0]);
      const uint32_t leader_full0 = ptx::map_to_cta(full0, 0);  // the rank lives in the upper address bits
      for (int tile = cluster; tile < total_tiles && ok; tile += num_clusters) {
        const TilePlan tp = plan_tile(P, tile, num_kb);
        const PairTile pt = tp.pt;
        const int r = static_cast<int>(rank);
        const int mat = tp.base_mat + of_rank(pt.dm, r);  // this CTA's matrix (its own A rows and B rows)
        const bool hh = pt.half != 0;  // half height: this CTA stages 64 A rows of row block i[0]
        const int row0 = hh ? pt.i[0] * 128 + r * 64 : of_rank(pt.i, r) * 128;
        const int half = 64 * pt.nbw;  // B rows (N columns) staged by each CTA
        const int b0 = pt.nbw == 2 ? of_rank(pt.j, r) * 128 : pt.j[0] * 128 + r * 64;
        const uint32_t stage_tx = 2u * static_cast<uint32_t>((hh ? kTileABytes / 2 : kTileABytes) + half * 128);
        const int kb_a = tp.kb_a, kb_b = tp.kb_b;
        // a transposed-formulation tile takes its operands from the other two 64 x 64 maps
        const CUtensorMap* map_a64 = tp.swapped ? &P.map_b : &P.map_a64;
        const CUtensorMap* map_b = tp.swapped ? &P.map_a64 : &P.map_b;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = ptx::mbar_wait(empty0 + stage * 8, phase ^ 1u, abort_flag);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) {
            if (elected) report_timeout(P, mat);
            break;
          }
          if (elected) {
            const uint32_t leader_full = leader_full0 + stage * 8;
            const uint32_t sa = ring_u32 + stage * kStageBytes;
            const uint32_t sb = sa + kTileABytes;
            const int k0 = kb * kBK;
            if (rank == 0) ptx::mbar_arrive_expect_tx(full0 + stage * 8, stage_tx);
            if (kb >= kb_a) {
              // K-major; the 64 x 64 box gives the first 64 rows of the 128-row tile's layout
              if (hh) ptx::tma_load_3d_pair(sa, map_a64, k0, row0, mat, leader_full);
              else ptx::tma_load_3d_pair(sa, &P.map_a, k0, row0, mat, leader_full);
            } else {
              ptx::tma_load_3d_pair(sa, map_a64, row0, k0, mat, leader_full);
              if (!hh) ptx::tma_load_3d_pair(sa + 8192, map_a64, row0 + 64, k0, mat, leader_full);
            }
            if (kb >= kb_b) {
              ptx::tma_load_3d_pair(sb, map_b, k0, b0, mat, leader_full);
              if (pt.nbw == 2) ptx::tma_load_3d_pair(sb + 8192, map_b, k0, b0 + 64, mat, leader_full);
            } else {
              ptx::tma_load_3d_pair(sb, map_b, b0, k0, mat, leader_full);
              if (pt.nbw == 2) ptx::tma_load_3d_pair(sb + 8192, map_b, b0 + 64, k0, mat, leader_full);
            }
          }
          __syncwarp();
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);  // let copies in flight land
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------- UMMA issuer (leader CTA) ----
    // The issuing thread is the pacemaker of the tensor pipe, so its loop is
    // kept short: the shared-memory descriptors differ only in the low word
    // (encoded start address), which advances by a constant per K = 16 step.
    // The whole warp walks the loop, so the operands of the UMMA instructions are
    // warp-uniform values; one elected lane issues them and their commits.
    if (rank == 0) {
      const bool elected = ptx::elect_one();
      uint32_t stage = 0, phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint32_t ring_enc = ptx::smem_u32(ring) >> 4;
      const uint32_t full0 = ptx::smem_u32(&bars->full[0]);
      const uint32_t empty0 = ptx::smem_u32(&bars->empty[0]);
      constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024, version 1, 128B swizzle
      constexpr uint32_t kLboK = (16u >> 4) << 16;      // K-major: LBO 16
      constexpr uint32_t kLboMN = (8192u >> 4) << 16;   // MN-major: LBO 8192 (next 64-element chunk)
      for (int tile = cluster; tile < total_tiles && ok; tile += num_clusters) {
        const TilePlan tp = plan_tile(P, tile, num_kb);
        const PairTile pt = tp.pt;
        const int mat = tp.base_mat;
        const int kb_a = tp.kb_a, kb_b = tp.kb_b;
        ok = ptx::mbar_wait(ptx::smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) {
          if (elected) report_timeout(P, mat);
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kAccCols);
        uint32_t accumulate = 0;
        // up to three runs of K blocks, each with one operand layout
        const int cut1 = min(kb_a, kb_b), cut2 = max(kb_a, kb_b);
        int kb = 0;
#pragma unroll 1
        for (int seg = 0; seg < 3 && ok; ++seg) {
          const int seg_end = seg == 0 ? cut1 : (seg == 1 ? cut2 : num_kb);
          if (kb >= seg_end) continue;
          const bool a_mn = kb < kb_a, b_mn = kb < kb_b;
          const uint32_t idesc = ptx::make_idesc_bf16(pt.half ? 128 : 256, 128 * pt.nbw, a_mn ? 1 : 0, b_mn ? 1 : 0);
          const uint32_t a_fix = a_mn ? kLboMN : kLboK, b_fix = (b_mn ? kLboMN : kLboK) + (kTileABytes >> 4);
          const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4), b_step = b_mn ? (2048u >> 4) : (32u >> 4);
#pragma unroll 1
          for (; kb < seg_end; ++kb) {
            ok = ptx::mbar_wait(full0 + stage * 8, phase, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) {
              if (elected) report_timeout(P, mat);
              break;
            }
            ptx::tc_fence_after();
            const uint32_t enc = ring_enc + stage * (kStageBytes >> 4);
            const uint32_t a_lo = enc + a_fix, b_lo = enc + b_fix;
            if (elected) {
              ptx::umma_bf16_pair_lohi(d_tmem, a_lo, b_lo, kDescHi, idesc, accumulate);
              ptx::umma_bf16_pair_lohi(d_tmem, a_lo + a_step, b_lo + b_step, kDescHi, idesc, 1u);
              ptx::umma_bf16_pair_lohi(d_tmem, a_lo + 2 * a_step, b_lo + 2 * b_step, kDescHi, idesc, 1u);
              ptx::umma_bf16_pair_lohi(d_tmem, a_lo + 3 * a_step, b_lo + 3 * b_step, kDescHi, idesc, 1u);
              ptx::umma_commit_pair(empty0 + stage * 8, 3);
            }
            __syncwarp();
            accumulate = 1u;
            if (++stage == kStages) {
              stage = 0;
              phase ^= 1u;
            }
          }
        }
        if (!ok) break;
        if (elected) ptx::umma_commit_pair(ptx::smem_u32(&bars->acc_full[acc]), 3);
        __syncwarp();
        if (++acc == kNumAcc) {
          acc = 0;
          acc_phase ^= 1u;
        }
      }
    }
  } else {
    // ----------------------------------------------------------- epilogue ----
    const int q = warp & 3;  // TMEM lane quarter this warp may read = its 32 rows of the tile
    const uint32_t my_base = ptx::smem_u32(s_epi + q * kSubsPerWarp * kEntryBytes);
    unsigned long long* my_bars = bars->io_ready[q];
    // Ring of staging entries, one buffer per quarter.
    constexpr uint32_t ring_len = kSubsPerWarp;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t gq = 0;  // quarters processed so far by this warp

    // Lane 0 only: the quarter whose ring entry is armed next (ring_len - 1 ahead).
    QuarterCursor pre;
    uint32_t pre_g = 0;
    bool pre_valid = false;
    int loads_in_flight = 0;
    auto pre_seek = [&]() {  // moves `pre` to a quarter, opening tiles as needed
      while (pre_valid && !pre.has_quarter()) {
        pre_valid = pre.open_tile(P, pre.tile + num_clusters, total_tiles, static_cast<int>(rank), q);
      }
    };
    // Arms ring entry pre_g % ring_len for quarter pre_g: starts the TMA loads of
    // its input tiles, or just marks the entry free to write when there are none.
    auto arm_next = [&]() {
      if (!pre_valid) return;
      const uint32_t e = pre_g % ring_len;
      const uint32_t bar = ptx::smem_u32(&my_bars[e]);
      const uint32_t buf = my_base + e * kEntryBytes;
      const int row0 = pre.row0;
      const int col0 = pre.col0(pre.quarter());
      if (row0 >= pre.row_limit) {  // this warp's rows lie beyond the matrix: nothing to fetch
        ptx::mbar_arrive(bar);
      } else if (P.last) {
        // the tile is in W's own orientation (see the header): W[row0.., col0..]
        ptx::mbar_arrive_expect_tx(bar, kEntryBytes);
        ptx::tma_load_3d(buf, P.wmaps + pre.mat, col0, row0, 0, bar);
        if (kWFp32) ptx::tma_load_3d(buf + kSubBytes, P.wmaps + pre.mat, col0 + 32, row0, 0, bar);
        ++loads_in_flight;
      } else if (P.has_in) {
        ptx::mbar_arrive_expect_tx(bar, kSubBytes);
        ptx::tma_load_3d(buf, &P.map_in, col0, row0, pre.mat, bar);
        ++loads_in_flight;
      } else {
        ptx::mbar_arrive(bar);
      }
      ++pre_g;
      pre.pop_quarter();
      pre_seek();
    };
    if (lane == 0) {
      pre_valid = pre.open_tile(P, cluster, total_tiles, static_cast<int>(rank), q);
      pre_seek();
      for (uint32_t i = 0; i + 1 < ring_len; ++i) arm_next();
    }

    QuarterCursor cur;
    bool ok = true;
    for (int tile = cluster; tile < total_tiles && ok; tile += num_clusters) {
      cur.open_tile(P, tile, total_tiles, static_cast<int>(rank), q);
      const int mat = cur.mat;
      ok = ptx::mbar_wait_relaxed(ptx::smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);  // the warp goes on or gives up as one
      if (!ok) {
        if (lane == 0) report_timeout(P, mat);
        break;
      }
      ptx::tc_fence_after();
      float o_sq = 0.f;  // last iteration: this lane's sum of O^2 over the tile
      if (cur.has_quarter()) {
        const MatScal sc = P.scal[mat];
        const float scale = P.scale_kind == 1 ? sc.inv_norm_sq : (P.scale_kind == 2 ? sc.inv_norm : 1.0f);
        const int row0 = cur.row0;  // first of this warp's rows
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * kAccCols) +
                               (static_cast<uint32_t>(q * 32) << 16);

        for (; cur.has_quarter() && ok; cur.pop_quarter(), ++gq) {
          const int qd = cur.quarter();
          const uint32_t e = gq % ring_len;
          const uint32_t buf = my_base + e * kEntryBytes;  // in / out (W on the last iteration)
          const int col0 = cur.col0(qd);
          // column of this lane's row that lies on the matrix diagonal, if the quarter holds it
          const bool diag_quarter = P.diag_add != 0.f && cur.col_block(qd) == cur.ib;
          const int dcol = row0 - cur.ib * 128 + lane - cur.col_in_block(qd);

          uint32_t v[64];
          ptx::tmem_ld_32x64(taddr + qd * 64, v);
          ok = ptx::mbar_wait(ptx::smem_u32(&my_bars[e]), (gq / ring_len) & 1u, abort_flag);
          ptx::tmem_ld_wait();
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) {
            if (lane == 0) report_timeout(P, mat);
            break;
          }

          if (!P.last) {
            // the diagonal add touches one element per row of a diagonal block's
            // quarter; the warp-uniform branch keeps it out of every other quarter
            auto combine = [&](auto with_diag) {
#pragma unroll
              for (int c8 = 0; c8 < 8; ++c8) {
                const uint32_t swz = static_cast<uint32_t>(lane * 128 + ((c8 ^ (lane & 7)) << 4));
                float in[8];
                if (P.has_in) {
                  uint32_t w0, w1, w2, w3;
                  lds128(buf + swz, w0, w1, w2, w3);
                  unpack8(w0, w1, w2, w3, in);
                } else {
#pragma unroll
                  for (int i = 0; i < 8; ++i) in[i] = 0.f;
                }
                float o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  o[i] = scale * fmaf(P.c_acc, __uint_as_float(v[c8 * 8 + i]), P.c_in * in[i]);
                  if (decltype(with_diag)::value && c8 * 8 + i == dcol) o[i] += P.diag_add;
                }
                sts128(buf + swz, pack2(o[0], o[1]), pack2(o[2], o[3]), pack2(o[4], o[5]), pack2(o[6], o[7]));
              }
            };
            if (diag_quarter) combine(std::true_type{});
            else combine(std::false_type{});
          } else if (kWFp32) {
            // the same update on fp32 weights: 16 chunks of four columns in two boxes;
            // the bf16 copy of the new weights, if the matrix has one, goes straight
            // from the registers to global memory (a 128-byte run per row and quarter,
            // in 32-byte stores where the row is aligned for them)
            const MatDesc& md = P.descs[mat];
            __nv_bfloat16* shadow = static_cast<__nv_bfloat16*>(md.w_shadow);
            const int w_cols = md.cols;
            const bool row_ok = row0 + lane < cur.row_limit && !sc.nonfinite;
            __nv_bfloat16* srow = shadow == nullptr ? nullptr
                                                    : shadow + static_cast<long long>(row0 + lane) * md.ld_ws + col0;
            // two 8-column chunks at a time: a 32-byte store per lane fills a whole sector
            const bool wide = srow != nullptr && ((reinterpret_cast<uintptr_t>(srow) & 31) == 0);
#pragma unroll
            for (int c16 = 0; c16 < 4; ++c16) {
              uint32_t packed[8];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const int c4 = 4 * c16 + h;
                const uint32_t addr = buf + static_cast<uint32_t>((c4 >> 3) * kSubBytes + lane * 128 +
                                                                  (((c4 & 7) ^ (lane & 7)) << 4));
                uint32_t w0, w1, w2, w3;
                lds128(addr, w0, w1, w2, w3);
                float w[4] = {__uint_as_float(w0), __uint_as_float(w1), __uint_as_float(w2), __uint_as_float(w3)};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const float o = scale * __uint_as_float(v[c4 * 4 + i]);
                  o_sq = fmaf(o, o, o_sq);
                  w[i] = fmaf(P.decay, w[i], P.upd_scale * o);
                }
                sts128(addr, __float_as_uint(w[0]), __float_as_uint(w[1]), __float_as_uint(w[2]), __float_as_uint(w[3]));
                packed[2 * h] = pack2(w[0], w[1]);
                packed[2 * h + 1] = pack2(w[2], w[3]);
              }
              if (srow != nullptr && row_ok) {
                const int c = col0 + c16 * 16;
                __nv_bfloat16* dst = srow + c16 * 16;
                if (wide && c + 16 <= w_cols) {
                  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(packed[0]),
                               "r"(packed[1]), "r"(packed[2]), "r"(packed[3]), "r"(packed[4]), "r"(packed[5]),
                               "r"(packed[6]), "r"(packed[7])
                               : "memory");
                } else {
#pragma unroll
                  for (int h8 = 0; h8 < 2; ++h8) {
                    if (c + 8 * h8 + 8 <= w_cols) {
                      *reinterpret_cast<uint4*>(dst + 8 * h8) =
                          make_uint4(packed[4 * h8], packed[4 * h8 + 1], packed[4 * h8 + 2], packed[4 * h8 + 3]);
                    } else {
                      for (int i = 0; i < 8 && c + 8 * h8 + i < w_cols; ++i) {
                        const uint32_t pr = packed[4 * h8 + (i >> 1)];
                        reinterpret_cast<unsigned short*>(dst + 8 * h8)[i] =
                            static_cast<unsigned short>((i & 1) ? (pr >> 16) : (pr & 0xFFFFu));
                      }
                    }
                  }
                }
              }
            }
          } else {
            // O = scale * acc;  W <- decay * W + upd_scale * O
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
              const uint32_t swz = static_cast<uint32_t>(lane * 128 + ((c8 ^ (lane & 7)) << 4));
              uint32_t w0, w1, w2, w3;
              float w[8];
              lds128(buf + swz, w0, w1, w2, w3);
              unpack8(w0, w1, w2, w3, w);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float o = scale * __uint_as_float(v[c8 * 8 + i]);
                o_sq = fmaf(o, o, o_sq);
                w[i] = fmaf(P.decay, w[i], P.upd_scale * o);
              }
              sts128(buf + swz, pack2(w[0], w[1]), pack2(w[2], w[3]), pack2(w[4], w[5]), pack2(w[6], w[7]));
            }
          }

          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (row0 >= cur.row_limit) {
              // rows beyond the matrix: nothing to store
            } else if (P.last) {
              if (!sc.nonfinite) {
                ptx::tma_store_3d(P.wmaps + mat, col0, row0, 0, buf);
                if (kWFp32 && col0 + 32 < P.descs[mat].cols)
                  ptx::tma_store_3d(P.wmaps + mat, col0 + 32, row0, 0, buf + kSubBytes);
              }
            } else {
              ptx::tma_store_3d(&P.map_out, col0, row0, mat, buf);
            }
            ptx::tma_store_commit();
            if (P.has_in && row0 < cur.row_limit) --loads_in_flight;
            ptx::tma_store_wait_read_all_but_one();  // every store but this quarter's has read its staging
            arm_next();                              // re-arms the entry of the previous quarter
          }
          __syncwarp();
        }
        if (!ok) break;
        if (row0 >= cur.row_limit) o_sq = 0.f;  // rows beyond the matrix were never loaded
      }
      if (P.last) {
        // Sum of O^2 of this warp's 32 rows of the tile (Algorithm 1 returns the
        // update RMS): fixed order within the lane, fixed butterfly across lanes;
        // one slot per (tile, CTA, warp), written even when it is zero.
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) o_sq += __shfl_xor_sync(0xFFFFFFFFu, o_sq, off);
        if (lane == 0) P.rms_partials[(static_cast<long long>(tile) * 2 + rank) * kEpiWarps + q] = o_sq;
      }
      // accumulator fully read: hand the TMEM stage back to the leader's issuer
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&bars->acc_empty[acc]), 0));
      }
      if (++acc == kNumAcc) {
        acc = 0;
        acc_phase ^= 1u;
      }
    }
    if (lane == 0) {
      ptx::tma_store_wait_all();
      if (loads_in_flight > 0) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);  // abort path: let input tiles in flight land
      }
    }
  }

  // ---------------------------------------------------------------- teardown --
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();  // the peer may still signal our barriers / read our tiles until here
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// Test probe for the bounded wait every kernel here relies on: one thread waits
// on an mbarrier that nothing ever arrives on, with a short limit, and records
// MUON_ERR_TIMEOUT exactly as the kernels do when a wait expires.  The wait
// ends by itself; nothing faults or hangs.
__global__ void wait_expiry_probe_kernel(DevStatus* status, int matrix_index, unsigned long long limit_ns) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
    if (!ptx::mbar_wait(ptx::smem_u32(&bar), 0u, &abort_flag, limit_ns)) {
      if (atomicCAS(&status->code, 0, -6 /* MUON_ERR_TIMEOUT */) == 0) status->matrix = matrix_index;
    }
  }
}

}  // namespace

cudaError_t launch_wait_expiry_probe(DevStatus* status, int matrix_index, unsigned long long limit_ns,
                                     cudaStream_t stream) {
  wait_expiry_probe_kernel<<<1, 32, 0, stream>>>(status, matrix_index, limit_ns);
  return cudaGetLastError();
}

namespace {

template <int kAccCols, int kStages, int kSubs, bool kWFp32 = false>
cudaError_t configure_one() {
  return cudaFuncSetAttribute(ns_gemm_kernel<kAccCols, kStages, kSubs, kWFp32>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                              smem_bytes(kStages, kSubs, kWFp32 ? kSubBytesFp32 : kSubBytes));
}

template <int kAccCols, int kStages, int kSubs, bool kWFp32 = false>
cudaError_t launch_one(const GemmParams& P, unsigned clusters, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters, 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes(kStages, kSubs, kWFp32 ? kSubBytesFp32 : kSubBytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // the kernel's set-up (barriers, TMEM allocation) may start while the previous kernel of the
  // stream drains; the kernel waits for that kernel's results itself (grid_dependency_wait)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, ns_gemm_kernel<kAccCols, kStages, kSubs, kWFp32>, P);
}

}  // namespace

cudaError_t gemm_configure() {
  cudaError_t e = configure_one<128, 4, 6>();
  if (e == cudaSuccess) e = configure_one<256, 4, 6>();
  if (e == cudaSuccess) e = configure_one<128, 5, 4>();
  if (e == cudaSuccess) e = configure_one<256, 5, 4>();
  if (e == cudaSuccess) e = configure_one<128, 4, 3, true>();
  if (e == cudaSuccess) e = configure_one<256, 4, 3, true>();
  return e;
}

// Largest number of co-resident CTA pairs (one CTA per SM).
cudaError_t gemm_max_clusters(int* out) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes(4, 6);
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(out, ns_gemm_kernel<256, 4, 6>, &cfg);
}

// acc_cols: 128 when every tile of the launch is one column block wide, else 256.
cudaError_t launch_ns_gemm(const GemmParams& P, int acc_cols, int max_clusters, cudaStream_t stream) {
  const long long total = static_cast<long long>(P.count / P.unit_mats) * P.tiles_per_unit +
                          (P.count % P.unit_mats ? P.tiles_per_tail : 0);
  if (total <= 0) return cudaSuccess;
  const unsigned clusters = static_cast<unsigned>(total < max_clusters ? total : max_clusters);
  const bool deep_ring = !P.has_in && !P.last;  // no epilogue input tiles: the Gram product
  if (deep_ring) {
    if (acc_cols == 128) return launch_one<128, 5, 4>(P, clusters, stream);
    return launch_one<256, 5, 4>(P, clusters, stream);
  }
  if (P.last && P.w_fp32) {  // same shared memory: three staging buffers of twice the size
    if (acc_cols == 128) return launch_one<128, 4, 3, true>(P, clusters, stream);
    return launch_one<256, 4, 3, true>(P, clusters, stream);
  }
  if (acc_cols == 128) return launch_one<128, 4, 6>(P, clusters, stream);
  return launch_one<256, 4, 6>(P, clusters, stream);
}

}  // namespace muon
