// Momentum / Nesterov / sum-of-squares / bf16 cast kernel, TMA-pipelined
// (Sec. 2.1: M <- mu*M + G; footnote 1: U = mu*M + G; ||U||_F accumulated per
// tile; bf16(U) stored short side first for the Newton-Schulz kernels).
//
// Persistent, one CTA per SM.  A matrix is cut into 64 x 64 tiles of its stored
// orientation; CTA c processes tiles c, c + grid, ... of the launch.
//   warp 8 (one lane)  producer: TMA loads of the G and M tiles kLookahead
//                      tiles ahead into a ring of kStages stages; when a tile
//                      is done it writes the tile's partial sum of squares and
//                      issues the TMA stores of the updated M tile (in place
//                      in shared memory) and of the bf16 tile (transposed in
//                      shared memory when rows > cols).
//   warps 0-7          arithmetic on the staged tiles, fp32; they synchronise
//                      with the producer through mbarriers only.
// HBM traffic is exactly G + M read, M + X written; everything is asynchronous
// bulk copies, so several tiles of loads and stores are in flight per SM.
//
// Used when every G and M of a bucket is TMA-addressable (16-byte aligned
// pointers and row pitches); momentum_cast_kernel is the general fallback.
// Every wait is bounded; on expiry the CTA records MUON_ERR_TIMEOUT and drains.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace muon {

namespace {

constexpr int kTile = 64;
constexpr int kComputeThreads = 256;
constexpr int kThreads = kComputeThreads + 32;
constexpr int kMBytes = kTile * kTile * 4;   // 16 KiB
constexpr int kXBytes = kTile * kTile * 2;   // 8 KiB

template <bool kGradFp32>
struct Cfg {
  static constexpr int kGBytes = kTile * kTile * (kGradFp32 ? 4 : 2);
  static constexpr int kStageBytes = kMBytes + kGBytes + kXBytes;
  static constexpr int kStages = kGradFp32 ? 5 : 6;
  static constexpr int kLookahead = kStages - 2;  // stores of two tiles may still be reading
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 1024;
};

struct TileInfo {
  int mat, row0, col0, transposed;
};

struct Ctrl {
  unsigned long long full[6];
  unsigned long long done[6];
  TileInfo info[6];
  float warp_sums[6][8];
  int abort_flag;
};
static_assert(sizeof(Ctrl) <= 1024, "control block too large");

__device__ __forceinline__ void stream_report_timeout(const StreamTmaParams& P, int mat) {
  if (atomicCAS(&P.status->code, 0, -6 /* MUON_ERR_TIMEOUT */) == 0) {
    P.status->matrix = P.descs[mat].global_index;
  }
}

template <bool kGradFp32>
__global__ void __launch_bounds__(kThreads, 1)
momentum_tma_kernel(const __grid_constant__ StreamTmaParams P) {
  using C = Cfg<kGradFp32>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + C::kStages * C::kStageBytes);
  volatile int* abort_flag = &ctrl->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long total = static_cast<long long>(P.count) * P.tiles_per_matrix;
  const int my_tiles = static_cast<int>((total - blockIdx.x + gridDim.x - 1) / gridDim.x);

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctrl->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctrl->done[s]), kComputeThreads / 32);
    }
    ctrl->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&P.map_x);
  }
  __syncthreads();

  if (warp == kComputeThreads / 32) {
    // ------------------------------------------------------------ producer ----
    if (lane == 0) {
      const int tiles_c_nt = (P.n + kTile - 1) / kTile, tiles_c_t = (P.m + kTile - 1) / kTile;
      auto issue_loads = [&](int i) {
        const int s = i % C::kStages;
        const long long t = blockIdx.x + static_cast<long long>(i) * gridDim.x;
        const int mat = static_cast<int>(t / P.tiles_per_matrix);
        const int ti = static_cast<int>(t - static_cast<long long>(mat) * P.tiles_per_matrix);
        const int tr_flag = P.descs[mat].transposed;
        // stored orientation: m x n (rows <= cols) or n x m (rows > cols)
        const int tiles_c = tr_flag ? tiles_c_t : tiles_c_nt;
        const int tr = ti / tiles_c, tc = ti - tr * tiles_c;
        TileInfo inf{mat, tr * kTile, tc * kTile, tr_flag};
        ctrl->info[s] = inf;
        const uint32_t bar = ptx::smem_u32(&ctrl->full[s]);
        const uint32_t base = ptx::smem_u32(smem + s * C::kStageBytes);
        ptx::mbar_arrive_expect_tx(bar, kMBytes + C::kGBytes);
        ptx::tma_load_3d(base, P.mmaps + mat, inf.col0, inf.row0, 0, bar);
        ptx::tma_load_3d(base + kMBytes, P.gmaps + mat, inf.col0, inf.row0, 0, bar);
      };
      int issued = 0;
      for (; issued < C::kLookahead && issued < my_tiles; ++issued) issue_loads(issued);
      bool ok = true;
      for (int i = 0; i < my_tiles; ++i) {
        const int s = i % C::kStages;
        const uint32_t phase = static_cast<uint32_t>(i / C::kStages) & 1u;
        if (!ptx::mbar_wait(ptx::smem_u32(&ctrl->done[s]), phase, abort_flag)) {
          stream_report_timeout(P, ctrl->info[s].mat);
          ok = false;
          break;
        }
        const TileInfo inf = ctrl->info[s];
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kComputeThreads / 32; ++w) sum += ctrl->warp_sums[s][w];
        const long long t = blockIdx.x + static_cast<long long>(i) * gridDim.x;
        P.partials[t] = sum;
        const uint32_t base = ptx::smem_u32(smem + s * C::kStageBytes);
        // a matrix whose gradient was found non-finite keeps its momentum (its norm comes out
        // non-finite all the same, so its weight is kept too)
        if (P.g_bad == nullptr || P.g_bad[inf.mat] == 0) ptx::tma_store_3d(P.mmaps + inf.mat, inf.col0, inf.row0, 0, base);
        if (inf.transposed) {
          ptx::tma_store_3d(&P.map_x, inf.row0, inf.col0, inf.mat, base + kMBytes + C::kGBytes);
        } else {
          ptx::tma_store_3d(&P.map_x, inf.col0, inf.row0, inf.mat, base + kMBytes + C::kGBytes);
        }
        ptx::tma_store_commit();
        if (issued < my_tiles) {
          // the stage of tile `issued` was last used by tile issued - kStages = i - 2
          ptx::tma_store_wait_read_all_but_two();
          issue_loads(issued);
          ++issued;
        }
      }
      ptx::tma_store_wait_all();
      if (!ok) {
        for (int k = 0; k < 64; ++k) __nanosleep(1000);  // let loads in flight land
      }
    }
  } else {
    // ---------------------------------------------------------- arithmetic ----
    const int tid = threadIdx.x;
    for (int i = 0; i < my_tiles; ++i) {
      const int s = i % C::kStages;
      const uint32_t phase = static_cast<uint32_t>(i / C::kStages) & 1u;
      bool ok = ptx::mbar_wait(ptx::smem_u32(&ctrl->full[s]), phase, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) {
        if (lane == 0) stream_report_timeout(P, 0);
        break;
      }
      const int transposed = ctrl->info[s].transposed;
      uint8_t* stage = smem + s * C::kStageBytes;
      float* mb = reinterpret_cast<float*>(stage);
      const uint8_t* gb = stage + kMBytes;
      const uint32_t xb = ptx::smem_u32(stage + kMBytes + C::kGBytes);
      float sumsq = 0.f;
      if (!transposed) {
        // thread: 4 consecutive columns of rows (tid / 16) + 16 p
        const int c4 = (tid & 15) * 4;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const int r = (tid >> 4) + 16 * p;
          float4 m4 = *reinterpret_cast<const float4*>(mb + r * kTile + c4);
          float g[4];
          if (kGradFp32) {
            const float4 g4 = *reinterpret_cast<const float4*>(gb + (r * kTile + c4) * 4);
            g[0] = g4.x; g[1] = g4.y; g[2] = g4.z; g[3] = g4.w;
          } else {
            const uint2 g2 = *reinterpret_cast<const uint2*>(gb + (r * kTile + c4) * 2);
            g[0] = __uint_as_float(g2.x << 16); g[1] = __uint_as_float(g2.x & 0xFFFF0000u);
            g[2] = __uint_as_float(g2.y << 16); g[3] = __uint_as_float(g2.y & 0xFFFF0000u);
          }
          float mm[4] = {m4.x, m4.y, m4.z, m4.w}, u[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            mm[e] = fmaf(P.mu, mm[e], g[e]);                       // M_t = mu*M_{t-1} + G
            u[e] = P.nesterov ? fmaf(P.mu, mm[e], g[e]) : mm[e];   // footnote 1
            sumsq = fmaf(u[e], u[e], sumsq);
          }
          *reinterpret_cast<float4*>(mb + r * kTile + c4) = make_float4(mm[0], mm[1], mm[2], mm[3]);
          __nv_bfloat162 h0 = __floats2bfloat162_rn(u[0], u[1]), h1 = __floats2bfloat162_rn(u[2], u[3]);
          const uint32_t addr = xb + r * 128 + ((((c4 >> 3) ^ (r & 7))) << 4) + (c4 & 7) * 2;
          asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t*>(&h0)),
                       "r"(*reinterpret_cast<uint32_t*>(&h1))
                       : "memory");
        }
      } else {
        // thread: column c of source rows 16 rq .. 16 rq + 15; the bf16 tile is
        // stored transposed (row c of the staged tile holds source column c)
        const int c = tid & 63, rq = tid >> 6;
        uint32_t packed[8];
#pragma unroll
        for (int e2 = 0; e2 < 8; ++e2) {
          float u2[2];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int r = rq * 16 + e2 * 2 + h;
            const float m_old = mb[r * kTile + c];
            float g;
            if (kGradFp32) g = *reinterpret_cast<const float*>(gb + (r * kTile + c) * 4);
            else g = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(gb + (r * kTile + c) * 2));
            const float mn = fmaf(P.mu, m_old, g);
            const float u = P.nesterov ? fmaf(P.mu, mn, g) : mn;
            sumsq = fmaf(u, u, sumsq);
            mb[r * kTile + c] = mn;
            u2[h] = u;
          }
          __nv_bfloat162 hh = __floats2bfloat162_rn(u2[0], u2[1]);
          packed[e2] = *reinterpret_cast<uint32_t*>(&hh);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const uint32_t addr = xb + c * 128 + ((((rq * 2 + j) ^ (c & 7))) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(packed[4 * j]),
                       "r"(packed[4 * j + 1]), "r"(packed[4 * j + 2]), "r"(packed[4 * j + 3])
                       : "memory");
        }
      }
      ptx::fence_proxy_async_smem();
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sumsq += __shfl_xor_sync(0xFFFFFFFFu, sumsq, o);
      __syncwarp();  // every lane's tile writes are ordered before lane 0's arrival
      if (lane == 0) {
        ctrl->warp_sums[s][warp] = sumsq;
        ptx::mbar_arrive(ptx::smem_u32(&ctrl->done[s]));
      }
      __syncwarp();
    }
  }
  __syncthreads();
}

}  // namespace

cudaError_t stream_tma_configure() {
  cudaError_t e = cudaFuncSetAttribute(momentum_tma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Cfg<false>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(momentum_tma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<true>::kSmemBytes);
}

cudaError_t launch_momentum_tma(const StreamTmaParams& P, bool grad_fp32, int num_sms, cudaStream_t stream) {
  const long long total = static_cast<long long>(P.count) * P.tiles_per_matrix;
  if (total <= 0) return cudaSuccess;
  const unsigned grid = static_cast<unsigned>(total < num_sms ? total : num_sms);
  if (grad_fp32) momentum_tma_kernel<true><<<grid, kThreads, Cfg<true>::kSmemBytes, stream>>>(P);
  else momentum_tma_kernel<false><<<grid, kThreads, Cfg<false>::kSmemBytes, stream>>>(P);
  return cudaGetLastError();
}

}  // namespace muon
