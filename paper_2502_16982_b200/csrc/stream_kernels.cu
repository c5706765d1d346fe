// HBM-streaming kernels of the Muon step:
//   momentum_cast_kernel : M <- mu*M + G, U = Nesterov blend or M, per-tile sum
//                          of U^2, bf16(U) stored short side first (transposed
//                          when rows > cols)                    (Sec. 2.1 rule
//                          line 1, footnote 1, Newton-Schulz paragraph)
//   norm_finalise_kernel : fixed-order sum of the per-tile partials ->
//                          ||U||_F, 1/(||U||_F + eps), non-finite flag
//   update_from_x_kernel : the weight update from a stored O (ns_steps == 0,
//                          where O = X0; fp32 weights; weights that a TMA
//                          descriptor cannot address)
// The division by the norm is deferred: bf16(U) is stored un-normalised and the
// scalar 1/(||U||_F+eps) is applied in fp32 by the first iteration's epilogues.
#include <cuda_bf16.h>

#include "internal.h"

namespace muon {

namespace {

constexpr int kRowStep = kStreamThreads / 16;        // rows covered by one pass of the CTA
constexpr int kRowsPerThread = kSTR / kRowStep;      // passes
static_assert(kRowsPerThread * kRowStep == kSTR, "tile rows must be a multiple of the pass");

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
  return __uint_as_float(bits16 << 16);
}

template <bool kGradFp32>
__device__ __forceinline__ void load_g8(const void* g, long long off, bool vec, int valid,
                                        float (&out)[8]) {
  if (kGradFp32) {
    const float* p = reinterpret_cast<const float*>(g) + off;
    if (vec && valid == 8) {
      float4 a = __ldcs(reinterpret_cast<const float4*>(p));
      float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
      out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
      out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) out[e] = e < valid ? p[e] : 0.f;
    }
  } else {
    const __nv_bfloat16* p = reinterpret_cast<const __nv_bfloat16*>(g) + off;
    if (vec && valid == 8) {
      uint4 a = __ldcs(reinterpret_cast<const uint4*>(p));
      out[0] = bf16_bits_to_float(a.x & 0xFFFFu); out[1] = bf16_bits_to_float(a.x >> 16);
      out[2] = bf16_bits_to_float(a.y & 0xFFFFu); out[3] = bf16_bits_to_float(a.y >> 16);
      out[4] = bf16_bits_to_float(a.z & 0xFFFFu); out[5] = bf16_bits_to_float(a.z >> 16);
      out[6] = bf16_bits_to_float(a.w & 0xFFFFu); out[7] = bf16_bits_to_float(a.w >> 16);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) out[e] = e < valid ? __bfloat162float(p[e]) : 0.f;
    }
  }
}

// One CTA = one kSTR x kSTC (64 x 128) tile of one matrix in its stored
// orientation.  Thread t owns 8 consecutive columns (t % 16) of rows
// (t / 16) + 32*p, p = 0..1; two rows per thread keep the register count low
// enough for two 512-thread CTAs per SM.
template <bool kGradFp32>
__global__ void __launch_bounds__(kStreamThreads, 2)
momentum_cast_kernel(const StreamParams P) {
  // bf16 tile for the transposed store; +2 elements of row padding keeps the
  // column reads off a single bank.
  __shared__ __nv_bfloat16 tile[kSTR][kSTC + 2];
  __shared__ float warp_sums[kStreamThreads / 32];

  const int mat = blockIdx.x / P.tiles_per_matrix;
  const int t_in = blockIdx.x - mat * P.tiles_per_matrix;
  const MatDesc d = P.descs[mat];
  const int tiles_c = (d.cols + kSTC - 1) / kSTC;
  const int tiles_r = (d.rows + kSTR - 1) / kSTR;
  float* partial = P.partials + static_cast<long long>(mat) * P.tiles_per_matrix + t_in;
  if (t_in >= tiles_c * tiles_r) {  // padding CTA (orientations differ in tile count)
    if (threadIdx.x == 0) *partial = 0.f;
    return;
  }
  const int tr = t_in / tiles_c, tc = t_in - tr * tiles_c;
  const int row0 = tr * kSTR, col0 = tc * kSTC;
  const int cgrp = threadIdx.x & 15, rsub = threadIdx.x >> 4;
  const int col = col0 + cgrp * 8;
  const int valid = min(8, max(0, d.cols - col));
  const bool vec = d.vec_ok != 0;
  const bool keep_m = P.g_bad != nullptr && P.g_bad[mat] != 0;

  float g[kRowsPerThread][8], m[kRowsPerThread][8];
#pragma unroll
  for (int p = 0; p < kRowsPerThread; ++p) {
    const int row = row0 + rsub + kRowStep * p;
    const bool in = row < d.rows && valid > 0;
    if (in) {
      load_g8<kGradFp32>(d.g, static_cast<long long>(row) * d.ld_g + col, vec, valid, g[p]);
      const float* mp = d.m + static_cast<long long>(row) * d.ld_m + col;
      if (vec && valid == 8) {
        float4 a = __ldcs(reinterpret_cast<const float4*>(mp));
        float4 b = __ldcs(reinterpret_cast<const float4*>(mp) + 1);
        m[p][0] = a.x; m[p][1] = a.y; m[p][2] = a.z; m[p][3] = a.w;
        m[p][4] = b.x; m[p][5] = b.y; m[p][6] = b.z; m[p][7] = b.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) m[p][e] = e < valid ? mp[e] : 0.f;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) { g[p][e] = 0.f; m[p][e] = 0.f; }
    }
  }

  // X is stored short side first: a row-major copy of U when rows <= cols,
  // its transpose otherwise.
  __nv_bfloat16* direct = d.transposed ? nullptr : P.x;
  __nv_bfloat16* transp = d.transposed ? P.x : nullptr;
  const long long direct_stride = P.x_stride, transp_stride = P.x_stride;
  const int ld_direct = P.ldx, ld_transp = P.ldx;

  float sumsq = 0.f;
#pragma unroll
  for (int p = 0; p < kRowsPerThread; ++p) {
    const int row = row0 + rsub + kRowStep * p;
    const bool in = row < d.rows && valid > 0;
    float u[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float mn = fmaf(P.mu, m[p][e], g[p][e]);  // M_t = mu*M_{t-1} + G
      m[p][e] = mn;
      u[e] = P.nesterov ? fmaf(P.mu, mn, g[p][e]) : mn;  // footnote 1
      sumsq = fmaf(u[e], u[e], sumsq);
    }
    __nv_bfloat162 h[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) h[e] = __floats2bfloat162_rn(u[2 * e], u[2 * e + 1]);
    if (in) {
      float* mp = d.m + static_cast<long long>(row) * d.ld_m + col;
      if (keep_m) {
        // a matrix whose gradient was found non-finite keeps its momentum
      } else if (vec && valid == 8) {
        __stcs(reinterpret_cast<float4*>(mp), make_float4(m[p][0], m[p][1], m[p][2], m[p][3]));
        __stcs(reinterpret_cast<float4*>(mp) + 1, make_float4(m[p][4], m[p][5], m[p][6], m[p][7]));
      } else {
        for (int e = 0; e < valid; ++e) mp[e] = m[p][e];
      }
      if (direct != nullptr) {
        __nv_bfloat16* xp = direct + mat * direct_stride + static_cast<long long>(row) * ld_direct + col;
        if (valid == 8) {  // workspace rows are 16-byte aligned by construction
          *reinterpret_cast<uint4*>(xp) = *reinterpret_cast<const uint4*>(h);
        } else {
          const __nv_bfloat16* hs = reinterpret_cast<const __nv_bfloat16*>(h);
          for (int e = 0; e < valid; ++e) xp[e] = hs[e];
        }
      }
    }
    if (transp != nullptr) {
      const int lr = rsub + kRowStep * p;
      __nv_bfloat162* trow = reinterpret_cast<__nv_bfloat162*>(&tile[lr][cgrp * 8]);
#pragma unroll
      for (int e = 0; e < 4; ++e) trow[e] = h[e];
    }
  }

  // Block reduction of the sum of squares in a fixed order.
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sumsq += __shfl_xor_sync(0xFFFFFFFFu, sumsq, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = sumsq;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kStreamThreads / 32; ++w) s += warp_sums[w];
    *partial = s;
  }

  if (transp != nullptr) {
    // Transposed store: output row = source column.  Each thread gathers 8
    // source rows of one column and writes 16 bytes; 8 threads cover the 64
    // source rows (128 bytes) of one output row.
    __nv_bfloat16* base = transp + mat * transp_stride;
    const int rgrp = threadIdx.x & 7;
    for (int c = threadIdx.x >> 3; c < kSTC; c += kStreamThreads / 8) {
      const int gcol = col0 + c;
      if (gcol >= d.cols) break;
      const int grow = row0 + rgrp * 8;
      if (grow >= d.rows) continue;
      __align__(16) __nv_bfloat16 v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = tile[rgrp * 8 + e][c];
      __nv_bfloat16* op = base + static_cast<long long>(gcol) * ld_transp + grow;
      const int nv = min(8, d.rows - grow);
      if (nv == 8) {
        *reinterpret_cast<uint4*>(op) = *reinterpret_cast<const uint4*>(v);
      } else {
        for (int e = 0; e < nv; ++e) op[e] = v[e];
      }
    }
  }
}

// One warp per matrix: sums the per-tile partials in a fixed order (lane-strided
// sequential accumulation, then a fixed butterfly), so the result is
// reproducible bit for bit.
__global__ void norm_finalise_kernel(const float* __restrict__ partials, int tiles_per_matrix,
                                     int count, float eps, const MatDesc* __restrict__ descs,
                                     MatScal* __restrict__ scal, float* __restrict__ norms,
                                     DevStatus* status) {
  const int mat = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (mat >= count) return;
  const int lane = threadIdx.x & 31;
  const float* p = partials + static_cast<long long>(mat) * tiles_per_matrix;
  float s = 0.f;
  for (int i = lane; i < tiles_per_matrix; i += 32) s += p[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) {
    const float nu = sqrtf(s);
    MatScal r;
    r.norm = nu;
    r.nonfinite = isfinite(nu) ? 0 : 1;
    const float inv = 1.0f / (nu + eps);
    r.inv_norm = r.nonfinite ? 0.f : inv;
    r.inv_norm_sq = r.nonfinite ? 0.f : inv * inv;
    scal[mat] = r;
    const int gidx = descs[mat].global_index;
    norms[gidx] = nu;
    if (r.nonfinite) {
      if (atomicCAS(&status->code, 0, -7 /* MUON_ERR_NONFINITE */) == 0) {
        status->matrix = gidx;
      }
    }
  }
}

// W <- decay*W + f*O with O = x (short side first, transposed back when rows >
// cols), f = -lr * (per-matrix update factor).  One CTA per 64 x 64 tile of W;
// the O tile passes through shared memory so that both the read of x and the
// accesses to W are coalesced in either orientation.  Optionally also writes a
// bf16 copy of the new fp32 weights (w_shadow).
template <bool kWFp32>
__global__ void __launch_bounds__(256)
update_from_x_kernel(const MatDesc* __restrict__ descs, const MatScal* __restrict__ scal,
                     const float* __restrict__ factors, const __nv_bfloat16* __restrict__ x,
                     long long x_stride, int ldx, float neg_lr, float decay) {
  __shared__ float tile[64][65];
  const int mat = blockIdx.y;
  const MatDesc d = descs[mat];
  if (scal[mat].nonfinite) return;
  const int tiles_c = (d.cols + 63) / 64;
  const int tr = blockIdx.x / tiles_c, tc = blockIdx.x - tr * tiles_c;
  if (tr * 64 >= d.rows) return;
  const int r0 = tr * 64, c0 = tc * 64;
  const float f = neg_lr * factors[mat];
  const __nv_bfloat16* xm = x + mat * x_stride;
  // x tile: rows (short side) xr0.., columns (long side) xc0..
  const int xr0 = d.transposed ? c0 : r0, xc0 = d.transposed ? r0 : c0;
  const int x_rows = d.transposed ? d.cols : d.rows, x_cols = d.transposed ? d.rows : d.cols;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
#pragma unroll 4
  for (int i = ty; i < 64; i += 4) {
    const int xr = xr0 + i, xc = xc0 + tx;
    tile[i][tx] = (xr < x_rows && xc < x_cols) ? __bfloat162float(xm[static_cast<long long>(xr) * ldx + xc]) : 0.f;
  }
  __syncthreads();
  // thread: 4 consecutive columns of rows (t / 16) + 16 p
  const int c4 = (threadIdx.x & 15) * 4;
  const bool vec_w = d.vec_ok && (d.w_shadow == nullptr || ((reinterpret_cast<uintptr_t>(d.w_shadow) & 7) == 0 && d.ld_ws % 4 == 0));
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const int i = (threadIdx.x >> 4) + 16 * p;
    const int r = r0 + i, c = c0 + c4;
    if (r >= d.rows || c >= d.cols) continue;
    float o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) o[e] = d.transposed ? tile[c4 + e][i] : tile[i][c4 + e];
    const long long off = static_cast<long long>(r) * d.ld_w + c;
    const int nv = min(4, d.cols - c);
    if (kWFp32) {
      float* w = reinterpret_cast<float*>(d.w) + off;
      __nv_bfloat16* sh = d.w_shadow ? reinterpret_cast<__nv_bfloat16*>(d.w_shadow) + static_cast<long long>(r) * d.ld_ws + c
                                     : nullptr;
      if (vec_w && nv == 4) {
        float4 w4 = *reinterpret_cast<const float4*>(w);
        w4.x = fmaf(decay, w4.x, f * o[0]);
        w4.y = fmaf(decay, w4.y, f * o[1]);
        w4.z = fmaf(decay, w4.z, f * o[2]);
        w4.w = fmaf(decay, w4.w, f * o[3]);
        *reinterpret_cast<float4*>(w) = w4;
        if (sh != nullptr) {
          __nv_bfloat162 h0 = __floats2bfloat162_rn(w4.x, w4.y), h1 = __floats2bfloat162_rn(w4.z, w4.w);
          *reinterpret_cast<uint2*>(sh) = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
        }
      } else {
        for (int e = 0; e < nv; ++e) {
          const float nw = fmaf(decay, w[e], f * o[e]);
          w[e] = nw;
          if (sh != nullptr) sh[e] = __float2bfloat16_rn(nw);
        }
      }
    } else {
      __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(d.w) + off;
      if (vec_w && nv == 4) {
        const uint2 w2 = *reinterpret_cast<const uint2*>(w);
        __nv_bfloat162 h0 = __floats2bfloat162_rn(fmaf(decay, __uint_as_float(w2.x << 16), f * o[0]),
                                                  fmaf(decay, __uint_as_float(w2.x & 0xFFFF0000u), f * o[1]));
        __nv_bfloat162 h1 = __floats2bfloat162_rn(fmaf(decay, __uint_as_float(w2.y << 16), f * o[2]),
                                                  fmaf(decay, __uint_as_float(w2.y & 0xFFFF0000u), f * o[3]));
        *reinterpret_cast<uint2*>(w) = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
      } else {
        for (int e = 0; e < nv; ++e) w[e] = __float2bfloat16_rn(fmaf(decay, __bfloat162float(w[e]), f * o[e]));
      }
    }
  }
}

// Update RMS (Algorithm 1, returned value) from per-matrix partial sums of O^2,
// one warp per matrix, fixed order: rms = |factor| * sqrt(sum / (rows * cols)).
// The sums come from the last Newton-Schulz epilogue or from sumsq_x_kernel; in
// the latter case (separate weight update) the kernel also leaves the factor
// the update kernel multiplies O by: `factor` * sn, or rms_target / RMS(O) * sn
// when the update is normalised (Sec. 3.1 "Update Norm"), with sn = 1/(||U||_F +
// eps) when the stored O is the un-normalised bf16(U) (no iteration).
__global__ void rms_finalise_kernel(const float* __restrict__ partials, int per_matrix, int count,
                                    float factor, const MatDesc* __restrict__ descs,
                                    const MatScal* __restrict__ scal, int use_inv_norm, float rms_target,
                                    int normalise, float* __restrict__ rms, float* __restrict__ factors) {
  const int mat = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (mat >= count) return;
  const int lane = threadIdx.x & 31;
  const float* p = partials + static_cast<long long>(mat) * per_matrix;
  float s = 0.f;
  for (int i = lane; i < per_matrix; i += 32) s += p[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) {
    const MatDesc d = descs[mat];
    const float sn = use_inv_norm ? scal[mat].inv_norm : 1.0f;
    const float o_rms = fabsf(sn) * sqrtf(s / (static_cast<float>(d.rows) * static_cast<float>(d.cols)));
    if (normalise) {
      rms[d.global_index] = o_rms > 0.f ? rms_target : 0.f;
      if (factors != nullptr) factors[mat] = o_rms > 0.f ? sn * rms_target / o_rms : 0.f;
    } else {
      rms[d.global_index] = fabsf(factor) * o_rms;
      if (factors != nullptr) factors[mat] = factor * sn;
    }
  }
}

// Partial sums of squares of a stored O (x, short side first, m x n): CTA
// (p, matrix) adds rows p, p + P, ... with 16-byte loads (rows of the workspace
// are 128-byte aligned) and a fixed reduction tree.
__global__ void __launch_bounds__(256)
sumsq_x_kernel(const __nv_bfloat16* __restrict__ x, long long x_stride, int ldx, int m, int n,
               float* __restrict__ partials) {
  __shared__ float warp_sums[8];
  const int mat = blockIdx.y;
  const __nv_bfloat16* xm = x + mat * x_stride;
  float s = 0.f;
  const int n8 = n / 8;
  for (int r = blockIdx.x; r < m; r += gridDim.x) {
    const __nv_bfloat16* row = xm + static_cast<long long>(r) * ldx;
    for (int c8 = threadIdx.x; c8 < n8; c8 += blockDim.x) {
      const uint4 v = *reinterpret_cast<const uint4*>(row + c8 * 8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xFFFF0000u);
        s = fmaf(lo, lo, s);
        s = fmaf(hi, hi, s);
      }
    }
    for (int c = n8 * 8 + threadIdx.x; c < n; c += blockDim.x) {
      const float v = __bfloat162float(row[c]);
      s = fmaf(v, v, s);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += warp_sums[w];
    partials[static_cast<long long>(mat) * gridDim.x + blockIdx.x] = t;
  }
}

// Makes the 128 x 128 diagonal blocks of a symmetric buffer symmetric bit for
// bit: element (r, c) below the diagonal takes the bits of (c, r).  The product
// kernels form a diagonal block in full, so for a product of two different
// matrices its two triangles differ by rounding; the consumers read the block
// both ways round, and the polynomial of the next iteration, whose terms nearly
// cancel, would magnify the difference.  One CTA per (block, matrix).
__global__ void __launch_bounds__(256)
symmetrise_diag_kernel(__nv_bfloat16* __restrict__ s, long long stride, int lda, int m) {
  // rows padded to 136 elements: 16-byte aligned for the vector stores, and a
  // column walk (stride 68 words) touches every bank once
  __shared__ __align__(16) unsigned short tile[128][136];
  unsigned short* base = reinterpret_cast<unsigned short*>(s) + blockIdx.y * stride;
  const int d0 = blockIdx.x * 128;
  const int size = min(128, m - d0);
  // 8-element chunks; rows are 16-byte aligned (lda is a multiple of 64) and
  // padded at least to the next multiple of 8 beyond m.  Thread t owns half a
  // row (8 chunks); all its loads are issued before the first is used.
  const int r = threadIdx.x >> 1, half = (threadIdx.x & 1) * 64;
  unsigned short* grow = base + static_cast<long long>(d0 + r) * lda + d0 + half;
  uint4 in[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c0 = half + k * 8;
    in[k] = make_uint4(0u, 0u, 0u, 0u);
    if (r < size && c0 < size && c0 + 7 >= r)  // holds elements on or above the diagonal
      in[k] = *reinterpret_cast<const uint4*>(grow + k * 8);
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) *reinterpret_cast<uint4*>(&tile[r][half + k * 8]) = in[k];
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c0 = half + k * 8;
    if (r < size && c0 < size && c0 < r) {  // holds elements below the diagonal
      unsigned short v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = c0 + e;
        v[e] = c < r ? tile[c][r] : tile[r][c];
      }
      uint4 out;
      out.x = v[0] | (static_cast<unsigned>(v[1]) << 16);
      out.y = v[2] | (static_cast<unsigned>(v[3]) << 16);
      out.z = v[4] | (static_cast<unsigned>(v[5]) << 16);
      out.w = v[6] | (static_cast<unsigned>(v[7]) << 16);
      *reinterpret_cast<uint4*>(grow + k * 8) = out;
    }
  }
}

}  // namespace

cudaError_t launch_symmetrise_diag(__nv_bfloat16* s, long long stride, int lda, int m, int count,
                                   cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  symmetrise_diag_kernel<<<dim3(static_cast<unsigned>((m + 127) / 128), static_cast<unsigned>(count)), 256, 0,
                           stream>>>(s, stride, lda, m);
  return cudaGetLastError();
}

cudaError_t launch_rms_finalise(const float* partials, int per_matrix, int count, float factor,
                                const MatDesc* descs, const MatScal* scal, bool use_inv_norm, float rms_target,
                                bool normalise, float* rms, float* factors, cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  const int warps = 4;
  rms_finalise_kernel<<<(count + warps - 1) / warps, warps * 32, 0, stream>>>(
      partials, per_matrix, count, factor, descs, scal, use_inv_norm ? 1 : 0, rms_target, normalise ? 1 : 0, rms,
      factors);
  return cudaGetLastError();
}

cudaError_t launch_sumsq_x(const __nv_bfloat16* x, long long x_stride, int ldx, int m, int n, int count,
                           int per_matrix, float* partials, cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  sumsq_x_kernel<<<dim3(static_cast<unsigned>(per_matrix), static_cast<unsigned>(count)), 256, 0, stream>>>(
      x, x_stride, ldx, m, n, partials);
  return cudaGetLastError();
}

// Optional pass before the momentum update: bad[mat] = 1 if the gradient of matrix `mat` holds an Inf
// or a NaN (exponent bits all ones), so that the momentum kernels can leave that matrix's M alone.
// Grid (row slabs, matrices); `bad` is zeroed before the launch.
template <bool kGradFp32>
__global__ void __launch_bounds__(256)
grad_finite_kernel(const MatDesc* __restrict__ descs, int* __restrict__ bad) {
  const int mat = blockIdx.y;
  const MatDesc d = descs[mat];
  const bool vec = (reinterpret_cast<uintptr_t>(d.g) & 15) == 0 && d.ld_g % 8 == 0;
  int found = 0;
  for (int row = blockIdx.x; row < d.rows; row += gridDim.x) {
    const long long base = static_cast<long long>(row) * d.ld_g;
    for (int c = threadIdx.x * 8; c < d.cols; c += blockDim.x * 8) {
      if (kGradFp32) {
        const uint32_t* p = reinterpret_cast<const uint32_t*>(d.g) + base + c;
        if (vec && c + 8 <= d.cols) {
          const uint4 a = *reinterpret_cast<const uint4*>(p), b = *(reinterpret_cast<const uint4*>(p) + 1);
          const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
          for (int e = 0; e < 8; ++e) found |= (w[e] & 0x7F800000u) == 0x7F800000u;
        } else {
          for (int e = 0; e < 8 && c + e < d.cols; ++e) found |= (p[e] & 0x7F800000u) == 0x7F800000u;
        }
      } else {
        const unsigned short* p = reinterpret_cast<const unsigned short*>(d.g) + base + c;
        if (vec && c + 8 <= d.cols) {
          const uint4 a = *reinterpret_cast<const uint4*>(p);
          const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
          for (int e = 0; e < 4; ++e)
            found |= ((w[e] & 0x7F80u) == 0x7F80u) | ((w[e] & 0x7F800000u) == 0x7F800000u);
        } else {
          for (int e = 0; e < 8 && c + e < d.cols; ++e) found |= (p[e] & 0x7F80u) == 0x7F80u;
        }
      }
    }
  }
  if (__syncthreads_or(found) && threadIdx.x == 0) bad[mat] = 1;
}

cudaError_t launch_grad_finite(const MatDesc* descs, int count, int rows_max, bool grad_fp32, int* bad,
                               cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(bad, 0, static_cast<size_t>(count) * sizeof(int), stream);
  if (e != cudaSuccess) return e;
  const dim3 grid(static_cast<unsigned>(rows_max < 64 ? rows_max : 64), static_cast<unsigned>(count));
  if (grad_fp32) grad_finite_kernel<true><<<grid, 256, 0, stream>>>(descs, bad);
  else grad_finite_kernel<false><<<grid, 256, 0, stream>>>(descs, bad);
  return cudaGetLastError();
}

cudaError_t launch_momentum_cast(const StreamParams& P, bool grad_fp32, cudaStream_t stream) {
  const unsigned grid = static_cast<unsigned>(P.count) * static_cast<unsigned>(P.tiles_per_matrix);
  if (grid == 0) return cudaSuccess;
  if (grad_fp32) momentum_cast_kernel<true><<<grid, kStreamThreads, 0, stream>>>(P);
  else momentum_cast_kernel<false><<<grid, kStreamThreads, 0, stream>>>(P);
  return cudaGetLastError();
}

cudaError_t launch_norm_finalise(const float* partials, int tiles_per_matrix, int count, float eps,
                                 const MatDesc* descs, MatScal* scal, float* norms,
                                 DevStatus* status, cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  const int warps = 4;
  norm_finalise_kernel<<<(count + warps - 1) / warps, warps * 32, 0, stream>>>(
      partials, tiles_per_matrix, count, eps, descs, scal, norms, status);
  return cudaGetLastError();
}

cudaError_t launch_update_from_x(const MatDesc* descs, const MatScal* scal, const float* factors,
                                 const __nv_bfloat16* x, long long x_stride, int ldx, int count, int m,
                                 int n, float neg_lr, float decay, bool w_fp32, cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  // both orientations of a bucket have the same number of 64 x 64 tiles
  dim3 grid(static_cast<unsigned>(((m + 63) / 64) * ((n + 63) / 64)), static_cast<unsigned>(count));
  if (w_fp32)
    update_from_x_kernel<true><<<grid, 256, 0, stream>>>(descs, scal, factors, x, x_stride, ldx, neg_lr, decay);
  else
    update_from_x_kernel<false><<<grid, 256, 0, stream>>>(descs, scal, factors, x, x_stride, ldx, neg_lr, decay);
  return cudaGetLastError();
}

}  // namespace muon
