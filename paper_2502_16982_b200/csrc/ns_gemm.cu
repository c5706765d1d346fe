// Newton-Schulz GEMM kernel for sm_100a (Eq. 2 of the paper, factored as
//   A = X X^T,  B = b*A + c*A*A,  X' = a*X + B*X):
// one persistent, warp-specialised kernel that serves all three products.
//
//   warp 0      TMA producer: streams 128x64 bf16 operand tiles into a
//               kStages-deep shared-memory ring (128-byte swizzle).
//   warp 1      UMMA issuer: tcgen05.mma (M=128, N=128, K=16, bf16 -> fp32)
//               into one of two TMEM accumulator stages; tcgen05.commit frees
//               ring slots and publishes finished accumulators.
//   warps 2-5   epilogue: tcgen05.ld the accumulator, combine with the input
//               tile (b*A, a*X) in fp32, round once to bf16, stage in shared
//               memory and TMA-store the tile and (for the symmetric products)
//               its mirror image; on the last iteration apply the scaled,
//               weight-decayed update to W instead (Sec. 2.2).
//
// Symmetric products compute only tiles with j >= i; the mirrored tile is the
// transpose of the same rounded values, so A and B are symmetric bit for bit,
// which is what makes A*A^T a valid way to form A^2.
//
// Every wait is bounded (ptx::mbar_wait).  On expiry the CTA raises its abort
// flag, records MUON_ERR_TIMEOUT in the device status word, lets copies in
// flight land, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace muon {

namespace {

constexpr int kTileABytes = kBM * kBK * 2;          // 16 KiB
constexpr int kTileBBytes = kBN * kBK * 2;          // 16 KiB
constexpr int kStageBytes = kTileABytes + kTileBBytes;
constexpr int kEpiIoBytes = 2 * kBM * 128;          // two 64-column halves, 128 rows x 128 B
constexpr int kEpiTBytes = kBN * kBM * 2;           // transposed bf16 tile / fp32 staging
constexpr int kNumAccStages = 2;
constexpr int kTmemCols = kNumAccStages * kBN;      // 256 fp32 columns
constexpr int kEpiThreads = 128;
constexpr int kFDirectPitch = 36;   // floats per row, 32-column fp32 staging (direct)
constexpr int kFTransPitch = 132;   // floats per row, 32-row fp32 staging (transposed)

struct SmemBarriers {
  unsigned long long full[kStages];
  unsigned long long empty[kStages];
  unsigned long long acc_full[kNumAccStages];
  unsigned long long acc_empty[kNumAccStages];
  unsigned long long in_full;
  uint32_t tmem_base;
  int abort_flag;
};

constexpr int kSmemBytes = 1024 /* alignment slack */ + kStages * kStageBytes + kEpiIoBytes +
                           kEpiTBytes + 256 /* barriers */;
static_assert(sizeof(SmemBarriers) <= 256, "barrier block too large");
static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB shared-memory limit");
static_assert(128 * kFDirectPitch * 4 <= kEpiTBytes, "fp32 staging (direct) too large");
static_assert(32 * kFTransPitch * 4 <= kEpiTBytes, "fp32 staging (transposed) too large");

struct TileCoord {
  int mat, i, j;
};

__device__ __forceinline__ TileCoord decode_tile(const GemmParams& P, int tile) {
  TileCoord t;
  t.mat = tile / P.tiles_per_matrix;
  int r = tile - t.mat * P.tiles_per_matrix;
  if (P.symmetric) {
    // upper triangle, row by row: row i holds nb - i tiles (j = i .. nb-1)
    int i = 0, len = P.nb_i;
    while (r >= len) {
      r -= len;
      --len;
      ++i;
    }
    t.i = i;
    t.j = i + r;
  } else {
    t.i = r / P.nb_j;
    t.j = r - t.i * P.nb_j;
  }
  return t;
}

__device__ __forceinline__ void report_timeout(const GemmParams& P, int mat) {
  if (atomicCAS(&P.status->code, 0, -6 /* MUON_ERR_TIMEOUT */) == 0) {
    P.status->matrix = P.descs[mat].global_index;
  }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

__global__ void __launch_bounds__(kGemmThreads, 1)
ns_gemm_kernel(const __grid_constant__ GemmParams P) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle atoms.
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* epi_io = smem + kStages * kStageBytes;
  uint8_t* epi_t = epi_io + kEpiIoBytes;
  SmemBarriers* bars = reinterpret_cast<SmemBarriers*>(epi_t + kEpiTBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_tiles = P.count * P.tiles_per_matrix;
  const int num_kb = (P.k + kBK - 1) / kBK;
  volatile int* abort_flag = &bars->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
    }
    for (int s = 0; s < kNumAccStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[s]), kEpiThreads / 32);
    }
    ptx::mbar_init(ptx::smem_u32(&bars->in_full), 1);
    bars->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&P.map_a);
    ptx::prefetch_tensormap(&P.map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&bars->tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------ TMA producer ----
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const TileCoord t = decode_tile(P, tile);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag)) {
            report_timeout(P, t.mat);
            ok = false;
            break;
          }
          const uint32_t bar = ptx::smem_u32(&bars->full[stage]);
          const uint32_t sa = ptx::smem_u32(ring + stage * kStageBytes);
          const uint32_t sb = sa + kTileABytes;
          ptx::mbar_arrive_expect_tx(bar, kStageBytes);
          ptx::tma_load_3d(sa, &P.map_a, kb * kBK, t.i * kBM, t.mat, bar);
          if (!P.b_mn_major) {
            ptx::tma_load_3d(sb, &P.map_b, kb * kBK, t.j * kBN, t.mat, bar);
          } else {
            // operand B read from the row-major K x N matrix: two boxes of
            // 64 (N) x 64 (K), each one 128-byte-swizzled atom column
            ptx::tma_load_3d(sb, &P.map_b, t.j * kBN, kb * kBK, t.mat, bar);
            ptx::tma_load_3d(sb + kTileBBytes / 2, &P.map_b, t.j * kBN + 64, kb * kBK, t.mat, bar);
          }
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        // let copies in flight land before the CTA's shared memory goes away
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------- UMMA issuer ----
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(kBM, kBN, 0, P.b_mn_major ? 1 : 0);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        if (!ptx::mbar_wait(ptx::smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag)) {
          report_timeout(P, tile / P.tiles_per_matrix);
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kBN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&bars->full[stage]), phase, abort_flag)) {
            report_timeout(P, tile / P.tiles_per_matrix);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(ring + stage * kStageBytes);
          const uint32_t sb = sa + kTileABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // K-major, 128-byte swizzle: 8-row groups 1024 B apart; a K step of
            // 16 elements is 32 bytes inside the swizzle atom.
            const uint64_t da = ptx::smem_desc_sw128(sa + k * 32, 16, 1024);
            // MN-major, 128-byte swizzle: 64-element N chunks 8192 B apart
            // (leading offset), 8-row K groups 1024 B apart (stride offset); a
            // K step of 16 rows is 2048 bytes.
            const uint64_t db = P.b_mn_major ? ptx::smem_desc_sw128(sb + k * 2048, 8192, 1024)
                                             : ptx::smem_desc_sw128(sb + k * 32, 16, 1024);
            ptx::umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(ptx::smem_u32(&bars->empty[stage]));
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        ptx::umma_commit(ptx::smem_u32(&bars->acc_full[acc]));
        if (++acc == kNumAccStages) {
          acc = 0;
          acc_phase ^= 1u;
        }
      }
    }
  } else {
    // ----------------------------------------------------------- epilogue ----
    const int q = warp & 3;            // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;       // tile row owned by this thread
    const int et = threadIdx.x - 64;   // 0..127 within the epilogue group
    const bool leader = (et == 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t in_phase = 0;
    const uint32_t io_base = ptx::smem_u32(epi_io);
    __nv_bfloat16* tbuf = reinterpret_cast<__nv_bfloat16*>(epi_t);
    float* fbuf = reinterpret_cast<float*>(epi_t);

    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const TileCoord t = decode_tile(P, tile);
      // staging buffers are free once the previous tile's stores have read them
      if (leader) ptx::tma_store_wait_read();
      ptx::named_bar_sync(1, kEpiThreads);
      if (P.has_in && leader) {
        const uint32_t bar = ptx::smem_u32(&bars->in_full);
        ptx::mbar_arrive_expect_tx(bar, kEpiIoBytes);
        ptx::tma_load_3d(io_base, &P.map_in, t.j * kBN, t.i * kBM, t.mat, bar);
        ptx::tma_load_3d(io_base + kEpiIoBytes / 2, &P.map_in, t.j * kBN + 64, t.i * kBM, t.mat, bar);
      }
      bool ok = ptx::mbar_wait(ptx::smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag);
      if (ok && P.has_in) {
        ok = ptx::mbar_wait(ptx::smem_u32(&bars->in_full), in_phase, abort_flag);
      }
      in_phase ^= 1u;
      // All 128 epilogue threads agree on whether to go on: a thread that gave
      // up must not leave the others waiting at a later barrier.
      if (ptx::named_bar_any(3, kEpiThreads, !ok)) {
        if (!ok) report_timeout(P, t.mat);
        break;
      }
      ptx::tc_fence_after();

      const MatScal sc = P.scal[t.mat];
      const float scale = P.scale_kind == 1 ? sc.inv_norm_sq : (P.scale_kind == 2 ? sc.inv_norm : 1.0f);
      const bool mirror = P.write_t && !(P.symmetric && t.i == t.j);
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * kBN) +
                             (static_cast<uint32_t>(q * 32) << 16);
      const MatDesc md = P.last ? P.descs[t.mat] : MatDesc{};

#pragma unroll 1
      for (int cc = 0; cc < kBN / 32; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(taddr + cc * 32, v);
        ptx::tmem_ld_wait();
        if (cc == kBN / 32 - 1) {
          // accumulator fully read: hand the TMEM stage back to the issuer
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->acc_empty[acc]));
        }
        const int half = cc >> 1;
        float o[32];
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          const int chunk = (cc & 1) * 4 + c8;  // 16-byte chunk within the 128-byte row
          const uint32_t saddr = io_base + half * (kEpiIoBytes / 2) + r * 128 +
                                 ((chunk ^ (r & 7)) << 4);
          float in[8];
          if (P.has_in) {
            uint32_t w0, w1, w2, w3;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                         : "r"(saddr));
            in[0] = __uint_as_float(w0 << 16); in[1] = __uint_as_float(w0 & 0xFFFF0000u);
            in[2] = __uint_as_float(w1 << 16); in[3] = __uint_as_float(w1 & 0xFFFF0000u);
            in[4] = __uint_as_float(w2 << 16); in[5] = __uint_as_float(w2 & 0xFFFF0000u);
            in[6] = __uint_as_float(w3 << 16); in[7] = __uint_as_float(w3 & 0xFFFF0000u);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) in[e] = 0.f;
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float a = __uint_as_float(v[c8 * 8 + e]);
            o[c8 * 8 + e] = scale * fmaf(P.c_acc, a, P.c_in * in[e]);
          }
          if (P.write_direct) {
            const uint32_t p0 = pack_bf16x2(o[c8 * 8 + 0], o[c8 * 8 + 1]);
            const uint32_t p1 = pack_bf16x2(o[c8 * 8 + 2], o[c8 * 8 + 3]);
            const uint32_t p2 = pack_bf16x2(o[c8 * 8 + 4], o[c8 * 8 + 5]);
            const uint32_t p3 = pack_bf16x2(o[c8 * 8 + 6], o[c8 * 8 + 7]);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(p0), "r"(p1),
                         "r"(p2), "r"(p3)
                         : "memory");
          }
          if (mirror) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              tbuf[(cc * 32 + c8 * 8 + e) * kBM + r] = __float2bfloat16_rn(o[c8 * 8 + e]);
            }
          }
        }

        if (P.last) {
          // Fused weight update for a 128 x 32 slab of O (Sec. 2.2):
          //   W <- (1 - lr*wd) * W - lr * rms_scale * sqrt(max(rows, cols)) * O
          // staged in fp32 in W's orientation, then applied with coalesced
          // accesses to W by all epilogue threads.
          if (!md.transposed) {
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              float4 f = make_float4(P.upd_scale * o[c4 * 4 + 0], P.upd_scale * o[c4 * 4 + 1],
                                     P.upd_scale * o[c4 * 4 + 2], P.upd_scale * o[c4 * 4 + 3]);
              *reinterpret_cast<float4*>(fbuf + r * kFDirectPitch + c4 * 4) = f;
            }
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c) fbuf[c * kFTransPitch + r] = P.upd_scale * o[c];
          }
          ptx::named_bar_sync(2, kEpiThreads);
          if (!sc.nonfinite) {
            // W-orientation slab: `srows` rows of `scols` columns
            const int srows = md.transposed ? 32 : 128;
            const int scols = md.transposed ? 128 : 32;
            const int pitch = md.transposed ? kFTransPitch : kFDirectPitch;
            const int grow0 = md.transposed ? t.j * kBN + cc * 32 : t.i * kBM;
            const int gcol0 = md.transposed ? t.i * kBM : t.j * kBN + cc * 32;
            const int tpr = scols / 4;  // threads per row, 4 elements each
            const int rpp = kEpiThreads / tpr;
            const int cl = (et % tpr) * 4;
            for (int rl = et / tpr; rl < srows; rl += rpp) {
              const int gr = grow0 + rl, gc = gcol0 + cl;
              if (gr >= md.rows || gc >= md.cols) continue;
              const float4 u = *reinterpret_cast<const float4*>(fbuf + rl * pitch + cl);
              const float uu[4] = {u.x, u.y, u.z, u.w};
              const int nv = min(4, md.cols - gc);
              const long long off = static_cast<long long>(gr) * md.ld_w + gc;
              if (P.w_fp32) {
                float* wp = reinterpret_cast<float*>(md.w) + off;
                if (md.vec_ok && nv == 4) {
                  float4 w = *reinterpret_cast<const float4*>(wp);
                  w.x = fmaf(P.decay, w.x, uu[0]); w.y = fmaf(P.decay, w.y, uu[1]);
                  w.z = fmaf(P.decay, w.z, uu[2]); w.w = fmaf(P.decay, w.w, uu[3]);
                  *reinterpret_cast<float4*>(wp) = w;
                } else {
                  for (int e = 0; e < nv; ++e) wp[e] = fmaf(P.decay, wp[e], uu[e]);
                }
              } else {
                __nv_bfloat16* wp = reinterpret_cast<__nv_bfloat16*>(md.w) + off;
                if (md.vec_ok && nv == 4) {
                  uint2 w = *reinterpret_cast<const uint2*>(wp);
                  const float w0 = __uint_as_float(w.x << 16), w1 = __uint_as_float(w.x & 0xFFFF0000u);
                  const float w2 = __uint_as_float(w.y << 16), w3 = __uint_as_float(w.y & 0xFFFF0000u);
                  w.x = pack_bf16x2(fmaf(P.decay, w0, uu[0]), fmaf(P.decay, w1, uu[1]));
                  w.y = pack_bf16x2(fmaf(P.decay, w2, uu[2]), fmaf(P.decay, w3, uu[3]));
                  *reinterpret_cast<uint2*>(wp) = w;
                } else {
                  for (int e = 0; e < nv; ++e)
                    wp[e] = __float2bfloat16_rn(fmaf(P.decay, __bfloat162float(wp[e]), uu[e]));
                }
              }
            }
          }
          ptx::named_bar_sync(2, kEpiThreads);
        }
      }

      if (P.write_direct || mirror) {
        ptx::fence_proxy_async_smem();
        ptx::named_bar_sync(2, kEpiThreads);
        if (leader) {
          if (P.write_direct) {
            ptx::tma_store_3d(&P.map_out, t.j * kBN, t.i * kBM, t.mat, io_base);
            ptx::tma_store_3d(&P.map_out, t.j * kBN + 64, t.i * kBM, t.mat, io_base + kEpiIoBytes / 2);
          }
          if (mirror) {
            ptx::tma_store_3d(&P.map_out_t, t.i * kBM, t.j * kBN, t.mat, ptx::smem_u32(epi_t));
          }
          ptx::tma_store_commit();
        }
      }
      if (++acc == kNumAccStages) {
        acc = 0;
        acc_phase ^= 1u;
      }
    }
    if (leader) ptx::tma_store_wait_all();
  }

  // ---------------------------------------------------------------- teardown --
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

cudaError_t gemm_configure() {
  return cudaFuncSetAttribute(ns_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t launch_ns_gemm(const GemmParams& P, int num_sms, cudaStream_t stream) {
  const long long total = static_cast<long long>(P.count) * P.tiles_per_matrix;
  if (total <= 0) return cudaSuccess;
  const unsigned grid = static_cast<unsigned>(total < num_sms ? total : num_sms);
  ns_gemm_kernel<<<grid, kGemmThreads, kSmemBytes, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace muon
