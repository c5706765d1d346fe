// Newton-Schulz GEMM kernel for sm_100a on CTA pairs (Eq. 2 of the paper,
// factored as  A = X X^T,  B = b*A + c*A*A,  X' = a*X + B*X).
//
// Two CTAs on neighbouring SMs form a cluster and share one UMMA
// (tcgen05.mma.cta_group::2): M = 256 (128 rows from each CTA's own A tile),
// N = 128 or 256 with the B operand split between the two CTAs' shared
// memories, so each CTA stages only half of B.  That halves the shared-memory
// and L2 bytes per FLOP compared with a 128x128 tile on one CTA.
//
// Per CTA (192 threads):
//   warp 0      TMA producer: its 128x64 A tile and its half of the B tile per
//               K block into a kStages-deep ring; byte counts of both CTAs are
//               reported to the leader CTA's "full" barrier.  No multicast.
//   warp 1      leader CTA only: UMMA issuer; tcgen05.commit (multicast to both
//               CTAs' barriers) frees ring slots and publishes accumulators.
//   warps 2-5   epilogue on the CTA's own 128 accumulator rows, 64 columns at a
//               time: tcgen05.ld, fp32 combine with the TMA-loaded input
//               (b*A, a*X), one bf16 rounding, swizzled staging, TMA store of
//               the block and, for the symmetric products, of its mirror image;
//               on the last iteration the scaled, weight-decayed update of W
//               (Sec. 2.2) instead.
//
// Symmetric products visit only column blocks j >= 2p of row pair p; the one
// below-diagonal block (2p+1, 2p) that the pair computes anyway is discarded
// and filled by the mirror of (2p, 2p+1), so A and B stay symmetric bit for bit.
//
// Every software wait is bounded (ptx::mbar_wait); on expiry the CTA records
// MUON_ERR_TIMEOUT, all roles drain, both CTAs meet at the final cluster
// barrier, TMEM is freed and the kernel returns.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace muon {

namespace {

constexpr int kPairStages = 5;
constexpr int kPTileABytes = 128 * kBK * 2;   // 16 KiB: this CTA's 128 A rows
constexpr int kPTileBBytes = 128 * kBK * 2;   // 16 KiB: up to 128 B rows (half of N = 256)
constexpr int kPStageBytes = kPTileABytes + kPTileBBytes;
constexpr int kQuarterBytes = 128 * 128;      // 128 rows x 64 bf16 columns
constexpr int kEpiThreads = 128;
constexpr int kNumAcc = 2;

struct PairBarriers {
  unsigned long long full[kPairStages];    // leader's copy is the live one
  unsigned long long empty[kPairStages];
  unsigned long long acc_full[kNumAcc];
  unsigned long long acc_empty[kNumAcc];   // leader's copy is the live one
  unsigned long long in_full[2];
  uint32_t tmem_base;
  int abort_flag;
};

constexpr int kPairSmemBytes = 1024 + kPairStages * kPStageBytes + 2 * kQuarterBytes /* input */ +
                               kQuarterBytes /* output */ + kQuarterBytes /* mirror / fp32 */ + 256;
static_assert(sizeof(PairBarriers) <= 256, "barrier block too large");
static_assert(kPairSmemBytes <= 232448, "exceeds the 227 KiB shared-memory limit");

__device__ __forceinline__ void pair_report_timeout(const PairGemmParams& P, int mat) {
  if (atomicCAS(&P.status->code, 0, -6 /* MUON_ERR_TIMEOUT */) == 0) {
    P.status->matrix = P.descs[mat].global_index;
  }
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// kAccCols: fp32 TMEM columns per accumulator stage = widest N (128 or 256).
template <int kAccCols>
__global__ void __launch_bounds__(kGemmThreads, 1)
ns_gemm_pair_kernel(const __grid_constant__ PairGemmParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* s_in = smem + kPairStages * kPStageBytes;
  uint8_t* s_out = s_in + 2 * kQuarterBytes;
  uint8_t* s_t = s_out + kQuarterBytes;
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(s_t + kQuarterBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();      // 0 = leader
  const int cluster = static_cast<int>(ptx::cluster_id_x());
  const int num_clusters = static_cast<int>(ptx::num_clusters_x());
  const int total_tiles = P.count * P.tiles_per_matrix;
  const int num_kb = (P.k + kBK - 1) / kBK;
  volatile int* abort_flag = &bars->abort_flag;
  constexpr uint32_t kTmemCols = kNumAcc * kAccCols;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
    }
    for (int s = 0; s < kNumAcc; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars->acc_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[s]), 2 * (kEpiThreads / 32));
    }
    ptx::mbar_init(ptx::smem_u32(&bars->in_full[0]), 1);
    ptx::mbar_init(ptx::smem_u32(&bars->in_full[1]), 1);
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
  if (P.debug != nullptr && threadIdx.x == 0) P.debug[blockIdx.x] = tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------ TMA producer ----
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = cluster; tile < total_tiles && ok; tile += num_clusters) {
        const int mat = tile / P.tiles_per_matrix;
        const PairTile pt = P.tiles[tile - mat * P.tiles_per_matrix];
        const int row0 = (2 * pt.p + static_cast<int>(rank)) * 128;
        const int half = 64 * pt.nbw;  // B rows (N columns) staged by each CTA
        const int b0 = pt.jb * 128 + static_cast<int>(rank) * half;
        const uint32_t stage_tx = 2u * static_cast<uint32_t>(kPTileABytes + half * 128);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag)) {
            pair_report_timeout(P, mat);
            ok = false;
            break;
          }
          const uint32_t local_full = ptx::smem_u32(&bars->full[stage]);
          const uint32_t leader_full = ptx::map_to_cta(local_full, 0);
          const uint32_t sa = ptx::smem_u32(ring + stage * kPStageBytes);
          const uint32_t sb = sa + kPTileABytes;
          if (rank == 0) ptx::mbar_arrive_expect_tx(local_full, stage_tx);
          ptx::tma_load_3d_pair(sa, &P.map_a, kb * kBK, row0, mat, leader_full);
          for (int h = 0; h < pt.nbw; ++h) {
            if (!P.b_mn_major) {
              ptx::tma_load_3d_pair(sb + h * 8192, &P.map_b, kb * kBK, b0 + 64 * h, mat, leader_full);
            } else {
              ptx::tma_load_3d_pair(sb + h * 8192, &P.map_b, b0 + 64 * h, kb * kBK, mat, leader_full);
            }
          }
          if (++stage == kPairStages) {
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
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = cluster; tile < total_tiles && ok; tile += num_clusters) {
        const int mat = tile / P.tiles_per_matrix;
        const PairTile pt = P.tiles[tile - mat * P.tiles_per_matrix];
        const uint32_t idesc = ptx::make_idesc_bf16(256, 128 * pt.nbw, 0, P.b_mn_major ? 1 : 0);
        if (!ptx::mbar_wait(ptx::smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag)) {
          pair_report_timeout(P, mat);
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kAccCols);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&bars->full[stage]), phase, abort_flag)) {
            pair_report_timeout(P, mat);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(ring + stage * kPStageBytes);
          const uint32_t sb = sa + kPTileABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            const uint64_t da = ptx::smem_desc_sw128(sa + k * 32, 16, 1024);
            const uint64_t db = P.b_mn_major ? ptx::smem_desc_sw128(sb + k * 2048, 8192, 1024)
                                             : ptx::smem_desc_sw128(sb + k * 32, 16, 1024);
            ptx::umma_bf16_pair(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit_pair(ptx::smem_u32(&bars->empty[stage]), 3);
          if (++stage == kPairStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        ptx::umma_commit_pair(ptx::smem_u32(&bars->acc_full[acc]), 3);
        if (++acc == kNumAcc) {
          acc = 0;
          acc_phase ^= 1u;
        }
      }
    }
  } else {
    // ----------------------------------------------------------- epilogue ----
    const int q = warp & 3;           // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;      // accumulator row owned by this thread
    const int et = threadIdx.x - 64;  // 0..127 within the epilogue group
    const bool leader = (et == 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    uint32_t in_phase[2] = {0u, 0u};
    const uint32_t in_base = ptx::smem_u32(s_in);
    const uint32_t out_base = ptx::smem_u32(s_out);
    __nv_bfloat16* tbuf = reinterpret_cast<__nv_bfloat16*>(s_t);
    float* fbuf = reinterpret_cast<float*>(s_t);
    bool aborted = false;
    uint32_t slab_ctr = 0;  // alternates the two fp32 staging buffers of the fused update

    for (int tile = cluster; tile < total_tiles && !aborted; tile += num_clusters) {
      const int mat = tile / P.tiles_per_matrix;
      const PairTile pt = P.tiles[tile - mat * P.tiles_per_matrix];
      const int ib = 2 * pt.p + static_cast<int>(rank);  // this CTA's row block
      const int row0 = ib * 128;
      const MatDesc md = P.descs[mat];
      const int out_rows = md.rows < md.cols ? md.rows : md.cols;  // m
      const int nq = 2 * pt.nbw;                                   // 64-column quarters in the tile
      int q_begin = 0;
      if (row0 >= out_rows) q_begin = nq;                         // ragged pair: nothing of ours
      else if (P.symmetric && pt.jb < ib) q_begin = 2;            // below-diagonal block: discard

      auto issue_input = [&](int qd) {
        const uint32_t bar = ptx::smem_u32(&bars->in_full[qd & 1]);
        ptx::mbar_arrive_expect_tx(bar, kQuarterBytes);
        ptx::tma_load_3d(in_base + (qd & 1) * kQuarterBytes, &P.map_in, pt.jb * 128 + qd * 64, row0, mat, bar);
      };
      if (P.has_in && leader) {
        if (q_begin < nq) issue_input(q_begin);
        if (q_begin + 1 < nq) issue_input(q_begin + 1);
      }
      bool ok = ptx::mbar_wait(ptx::smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag);
      // All 128 epilogue threads agree on whether to go on: a thread that gave
      // up must not leave the others waiting at a later barrier.
      if (ptx::named_bar_any(3, kEpiThreads, !ok)) {
        if (!ok) pair_report_timeout(P, mat);
        break;
      }
      ptx::tc_fence_after();
      const MatScal sc = P.scal[mat];
      const float scale = P.scale_kind == 1 ? sc.inv_norm_sq : (P.scale_kind == 2 ? sc.inv_norm : 1.0f);
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * kAccCols) +
                             (static_cast<uint32_t>(q * 32) << 16);

      for (int qd = q_begin; qd < nq; ++qd) {
        const int b = qd & 1;
        if (ok && P.has_in) {
          ok = ptx::mbar_wait(ptx::smem_u32(&bars->in_full[b]), in_phase[b], abort_flag);
          in_phase[b] ^= 1u;
        }
        if (leader) ptx::tma_store_wait_read();  // output and mirror staging are free again
        if (ptx::named_bar_any(3, kEpiThreads, !ok)) {  // uniform decision, as above
          if (!ok) pair_report_timeout(P, mat);
          aborted = true;
          break;
        }
        const int jblock = pt.jb + (qd >> 1);
        const bool mirror = P.symmetric && jblock > ib;
        const int col0 = jblock * 128 + (qd & 1) * 64;
        const uint32_t in_q = in_base + b * kQuarterBytes;

#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          // Last iteration: this thread's share of the W slab (8 groups of 4
          // consecutive elements), fetched early so the latency hides behind
          // the accumulator load and the staging.
          uint4 wreg[8];
          const int wrpp = md.transposed ? 4 : 16;                       // slab rows per pass
          const int wrl0 = md.transposed ? (et >> 5) : (et >> 3);        // first slab row
          const int wcl = (md.transposed ? (et & 31) : (et & 7)) * 4;    // slab column
          const int wgrow0 = md.transposed ? col0 + cc * 32 : row0;
          const int wgcol0 = md.transposed ? row0 : col0 + cc * 32;
          if (P.last && md.vec_ok && !sc.nonfinite) {
#pragma unroll
            for (int ps = 0; ps < 8; ++ps) {
              const int gr = wgrow0 + wrl0 + ps * wrpp, gc = wgcol0 + wcl;
              wreg[ps] = make_uint4(0u, 0u, 0u, 0u);
              if (gr < md.rows && gc + 4 <= md.cols) {
                const long long off = static_cast<long long>(gr) * md.ld_w + gc;
                if (P.w_fp32) {
                  wreg[ps] = *reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(md.w) + off);
                } else {
                  const uint2 t2 = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(md.w) + off);
                  wreg[ps].x = t2.x;
                  wreg[ps].y = t2.y;
                }
              }
            }
          }
          uint32_t v[32];
          ptx::tmem_ld_32x32(taddr + qd * 64 + cc * 32, v);
          ptx::tmem_ld_wait();
          float o[32];
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            const int chunk = cc * 4 + c8;  // 16-byte chunk within the 128-byte row
            const uint32_t swz = static_cast<uint32_t>(r * 128 + ((chunk ^ (r & 7)) << 4));
            float in[8];
            if (P.has_in) {
              uint32_t w0, w1, w2, w3;
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                           : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                           : "r"(in_q + swz));
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
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(out_base + swz),
                           "r"(pack2(o[c8 * 8 + 0], o[c8 * 8 + 1])), "r"(pack2(o[c8 * 8 + 2], o[c8 * 8 + 3])),
                           "r"(pack2(o[c8 * 8 + 4], o[c8 * 8 + 5])), "r"(pack2(o[c8 * 8 + 6], o[c8 * 8 + 7]))
                           : "memory");
            }
            if (mirror) {
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                tbuf[(cc * 32 + c8 * 8 + e) * 128 + r] = __float2bfloat16_rn(o[c8 * 8 + e]);
              }
            }
          }

          if (P.last) {
            // Fused weight update for a 128 x 32 slab of O (Sec. 2.2):
            //   W <- (1 - lr*wd) * W - lr * rms_scale * sqrt(max(rows, cols)) * O
            // O is staged in fp32 in W's orientation and applied with coalesced
            // accesses; W was fetched into registers before the accumulator load.
            float* fb = (!P.write_direct && (slab_ctr & 1)) ? reinterpret_cast<float*>(s_out) : fbuf;
            ++slab_ctr;
            if (!md.transposed) {
#pragma unroll
              for (int c = 0; c < 32; ++c) fb[r * 32 + (c ^ lane)] = P.upd_scale * o[c];
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) fb[c * 128 + r] = P.upd_scale * o[c];
            }
            ptx::named_bar_sync(2, kEpiThreads);
            if (!sc.nonfinite) {
#pragma unroll
              for (int ps = 0; ps < 8; ++ps) {
                const int rl = wrl0 + ps * wrpp;
                const int gr = wgrow0 + rl, gc = wgcol0 + wcl;
                if (gr >= md.rows || gc >= md.cols) continue;
                float uu[4];
                if (!md.transposed) {
#pragma unroll
                  for (int e = 0; e < 4; ++e) uu[e] = fb[rl * 32 + ((wcl + e) ^ (rl & 31))];
                } else {
                  const float4 u = *reinterpret_cast<const float4*>(fb + rl * 128 + wcl);
                  uu[0] = u.x; uu[1] = u.y; uu[2] = u.z; uu[3] = u.w;
                }
                const int nv = min(4, md.cols - gc);
                const long long off = static_cast<long long>(gr) * md.ld_w + gc;
                if (P.w_fp32) {
                  float* wp = reinterpret_cast<float*>(md.w) + off;
                  if (md.vec_ok && nv == 4) {
                    float4 w;
                    w.x = fmaf(P.decay, __uint_as_float(wreg[ps].x), uu[0]);
                    w.y = fmaf(P.decay, __uint_as_float(wreg[ps].y), uu[1]);
                    w.z = fmaf(P.decay, __uint_as_float(wreg[ps].z), uu[2]);
                    w.w = fmaf(P.decay, __uint_as_float(wreg[ps].w), uu[3]);
                    *reinterpret_cast<float4*>(wp) = w;
                  } else {
                    for (int e = 0; e < nv; ++e) wp[e] = fmaf(P.decay, wp[e], uu[e]);
                  }
                } else {
                  __nv_bfloat16* wp = reinterpret_cast<__nv_bfloat16*>(md.w) + off;
                  if (md.vec_ok && nv == 4) {
                    const uint32_t x = wreg[ps].x, y = wreg[ps].y;
                    uint2 w;
                    w.x = pack2(fmaf(P.decay, __uint_as_float(x << 16), uu[0]),
                                fmaf(P.decay, __uint_as_float(x & 0xFFFF0000u), uu[1]));
                    w.y = pack2(fmaf(P.decay, __uint_as_float(y << 16), uu[2]),
                                fmaf(P.decay, __uint_as_float(y & 0xFFFF0000u), uu[3]));
                    *reinterpret_cast<uint2*>(wp) = w;
                  } else {
                    for (int e = 0; e < nv; ++e)
                      wp[e] = __float2bfloat16_rn(fmaf(P.decay, __bfloat162float(wp[e]), uu[e]));
                  }
                }
              }
            }
            // with a single staging buffer (test tap on) wait before it is rewritten
            if (P.write_direct) ptx::named_bar_sync(2, kEpiThreads);
          }
        }

        if (P.write_direct || mirror) ptx::fence_proxy_async_smem();
        ptx::named_bar_sync(2, kEpiThreads);  // staging complete; input quarter fully read
        if (leader) {
          if (P.write_direct) ptx::tma_store_3d(&P.map_out, col0, row0, mat, out_base);
          if (mirror) ptx::tma_store_3d(&P.map_out_t, row0, col0, mat, ptx::smem_u32(s_t));
          if (P.write_direct || mirror) ptx::tma_store_commit();
          if (P.has_in && qd + 2 < nq) issue_input(qd + 2);
        }
      }
      if (aborted) break;
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
    if (leader) ptx::tma_store_wait_all();
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

}  // namespace

cudaError_t pair_gemm_configure() {
  cudaError_t e = cudaFuncSetAttribute(ns_gemm_pair_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kPairSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(ns_gemm_pair_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kPairSmemBytes);
}

// Largest number of co-resident CTA pairs (one CTA per SM).
cudaError_t pair_gemm_max_clusters(int acc_cols, int* out) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (acc_cols == 128) return cudaOccupancyMaxActiveClusters(out, ns_gemm_pair_kernel<128>, &cfg);
  return cudaOccupancyMaxActiveClusters(out, ns_gemm_pair_kernel<256>, &cfg);
}

cudaError_t launch_ns_gemm_pair(const PairGemmParams& P, int acc_cols, int max_clusters,
                                cudaStream_t stream) {
  const long long total = static_cast<long long>(P.count) * P.tiles_per_matrix;
  if (total <= 0) return cudaSuccess;
  const unsigned clusters = static_cast<unsigned>(total < max_clusters ? total : max_clusters);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * clusters, 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = kPairSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (acc_cols == 128) return cudaLaunchKernelEx(&cfg, ns_gemm_pair_kernel<128>, P);
  return cudaLaunchKernelEx(&cfg, ns_gemm_pair_kernel<256>, P);
}

}  // namespace muon
