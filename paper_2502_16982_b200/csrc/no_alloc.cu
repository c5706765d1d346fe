// muon_momentum_norm_static: momentum update and Frobenius norm of one matrix
// for callers that have no device memory to give as a workspace.
//
// The tile kernel below is a variant of the streaming momentum kernel: it
// updates M in place and leaves one partial sum of squares per 64 x 128 tile
// in scratch memory; a one-warp kernel then adds the partials in a fixed order.
// Here the scratch is not carved from a caller's workspace but lives in a
// file-scope __device__ array, which every GPU that loads this library holds
// from load until the process exits (kStaticScratchFloats * 4 bytes = 256 KiB).
//
// In host code the array's name only stands for the symbol; it is not a device
// address.  The address a kernel can use is looked up with
// cudaGetSymbolAddress, once per device and with that device current, the
// first time the entry point is called for that device.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <mutex>
#include <string>

#include "../../include/muon.h"

namespace muon {
void set_last_error(const char* msg);  // defined beside muon_last_error
}

namespace {

constexpr int kTileRows = 64;
constexpr int kTileCols = 128;
constexpr int kThreads = 512;
constexpr int kRowStep = kThreads / 16;            // rows per pass of the CTA
constexpr int kPasses = kTileRows / kRowStep;      // 2
constexpr int kStaticScratchFloats = MUON_STATIC_MAX_TILES;
constexpr int kMaxDevices = 64;

// Per-tile partial sums of squares.  Shared by every call on this GPU and never
// cleared: each call overwrites the entries of its own tiles before the
// finalising kernel reads exactly those entries, so nothing has to start at zero.
static __device__ __align__(256) float g_static_partials[kStaticScratchFloats];

std::mutex g_setup_mutex;
float* g_scratch_ptr[kMaxDevices] = {};  // device address of g_static_partials, per device

int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  muon::set_last_error(buf);
  return code;
}

template <bool kGradFp32>
__device__ __forceinline__ float load_g(const void* g, long long off) {
  if (kGradFp32) return reinterpret_cast<const float*>(g)[off];
  return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(g)[off]);
}

// One CTA per 64 x 128 tile; thread t owns 8 consecutive columns (t % 16) of
// rows (t / 16) and (t / 16) + 32.  M <- mu*M + G, U = mu*M + G (Nesterov-style)
// or M; the tile's sum of U^2 goes to partials[tile].
template <bool kGradFp32>
__global__ void __launch_bounds__(kThreads)
momentum_norm_static_kernel(const void* __restrict__ g, float* __restrict__ m, int rows, int cols,
                            long long ld_g, long long ld_m, float mu, int nesterov, int vec_ok,
                            float* __restrict__ partials) {
  __shared__ float warp_sums[kThreads / 32];
  const int tiles_c = (cols + kTileCols - 1) / kTileCols;
  const int tr = blockIdx.x / tiles_c, tc = blockIdx.x - tr * tiles_c;
  const int col = tc * kTileCols + (threadIdx.x & 15) * 8;
  const int valid = min(8, max(0, cols - col));
  float sumsq = 0.f;
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    const int row = tr * kTileRows + (threadIdx.x >> 4) + kRowStep * p;
    if (row >= rows || valid <= 0) continue;
    const long long og = static_cast<long long>(row) * ld_g + col;
    float* mp = m + static_cast<long long>(row) * ld_m + col;
    float gv[8], mv[8];
    if (vec_ok && valid == 8) {
      if (kGradFp32) {
        const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g) + og);
        const float4 b = *(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g) + og) + 1);
        gv[0] = a.x; gv[1] = a.y; gv[2] = a.z; gv[3] = a.w;
        gv[4] = b.x; gv[5] = b.y; gv[6] = b.z; gv[7] = b.w;
      } else {
        const uint4 a = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(g) + og);
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          gv[2 * e] = __uint_as_float(w[e] << 16);
          gv[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
        }
      }
      const float4 a = *reinterpret_cast<const float4*>(mp);
      const float4 b = *(reinterpret_cast<const float4*>(mp) + 1);
      mv[0] = a.x; mv[1] = a.y; mv[2] = a.z; mv[3] = a.w;
      mv[4] = b.x; mv[5] = b.y; mv[6] = b.z; mv[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        gv[e] = e < valid ? load_g<kGradFp32>(g, og + e) : 0.f;
        mv[e] = e < valid ? mp[e] : 0.f;
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float mn = fmaf(mu, mv[e], gv[e]);
      mv[e] = mn;
      const float u = nesterov ? fmaf(mu, mn, gv[e]) : mn;
      sumsq = fmaf(u, u, sumsq);
    }
    if (vec_ok && valid == 8) {
      *reinterpret_cast<float4*>(mp) = make_float4(mv[0], mv[1], mv[2], mv[3]);
      *(reinterpret_cast<float4*>(mp) + 1) = make_float4(mv[4], mv[5], mv[6], mv[7]);
    } else {
      for (int e = 0; e < valid; ++e) mp[e] = mv[e];
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sumsq += __shfl_xor_sync(0xFFFFFFFFu, sumsq, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = sumsq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) s += warp_sums[w];
    partials[blockIdx.x] = s;
  }
}

// One warp: lane-strided sequential sums, then a fixed butterfly.
__global__ void norm_static_finalise_kernel(const float* __restrict__ partials, int tiles,
                                            float* __restrict__ norm_out) {
  const int lane = threadIdx.x;
  float s = 0.f;
  for (int i = lane; i < tiles; i += 32) s += partials[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) *norm_out = sqrtf(s);
}

}  // namespace

extern "C" int muon_momentum_norm_static(const void* g, float* m, int rows, int cols, int64_t ld_g,
                                         int64_t ld_m, int g_dtype, float mu, int nesterov,
                                         float* norm_out, int device, void* stream_v) {
  if (!g || !m || !norm_out) return fail(MUON_ERR_INVALID_ARG, "g, m or norm_out is null");
  if (rows <= 0 || cols <= 0) return fail(MUON_ERR_INVALID_ARG, "rows and cols must be positive");
  if (ld_g < cols || ld_m < cols) return fail(MUON_ERR_INVALID_ARG, "leading dimension smaller than cols");
  if (g_dtype != MUON_DTYPE_BF16 && g_dtype != MUON_DTYPE_FP32)
    return fail(MUON_ERR_UNSUPPORTED, "g_dtype must be bf16 or fp32");
  if (device < 0 || device >= kMaxDevices) return fail(MUON_ERR_INVALID_ARG, "device ordinal out of range");
  const uintptr_t ga = g_dtype == MUON_DTYPE_FP32 ? 3 : 1;
  if ((reinterpret_cast<uintptr_t>(g) & ga) || (reinterpret_cast<uintptr_t>(m) & 3) ||
      (reinterpret_cast<uintptr_t>(norm_out) & 3))
    return fail(MUON_ERR_ALIGNMENT, "pointer not aligned to its element size");
  const long long tiles = static_cast<long long>((rows + kTileRows - 1) / kTileRows) *
                          ((cols + kTileCols - 1) / kTileCols);
  if (tiles > kStaticScratchFloats)
    return fail(MUON_ERR_UNSUPPORTED,
                "matrix of %d x %d needs %lld tiles of 64 x 128; the built-in scratch holds %d "
                "(use muon_step with a workspace for larger matrices)",
                rows, cols, tiles, kStaticScratchFloats);

  cudaError_t ce = cudaSetDevice(device);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(ce));
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[device] == nullptr) {
      // set-up, once per device: the device address behind the symbol
      void* p = nullptr;
      ce = cudaGetSymbolAddress(&p, g_static_partials);
      if (ce != cudaSuccess || p == nullptr)
        return fail(MUON_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(ce));
      g_scratch_ptr[device] = static_cast<float*>(p);
    }
    scratch = g_scratch_ptr[device];
  }

  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const bool ptr16 = ((reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(m)) & 15) == 0;
  const int vec_ok = (ptr16 && ld_g % 8 == 0 && ld_m % 8 == 0) ? 1 : 0;
  const unsigned grid = static_cast<unsigned>(tiles);
  if (g_dtype == MUON_DTYPE_FP32)
    momentum_norm_static_kernel<true><<<grid, kThreads, 0, stream>>>(g, m, rows, cols, ld_g, ld_m, mu,
                                                                      nesterov ? 1 : 0, vec_ok, scratch);
  else
    momentum_norm_static_kernel<false><<<grid, kThreads, 0, stream>>>(g, m, rows, cols, ld_g, ld_m, mu,
                                                                       nesterov ? 1 : 0, vec_ok, scratch);
  ce = cudaGetLastError();
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "momentum kernel launch: %s", cudaGetErrorString(ce));
  norm_static_finalise_kernel<<<1, 32, 0, stream>>>(scratch, static_cast<int>(tiles), norm_out);
  ce = cudaGetLastError();
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, "norm kernel launch: %s", cudaGetErrorString(ce));
  return MUON_OK;
}
