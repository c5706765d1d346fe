// Fused multi-tensor AdamW step for the parameters Muon does not handle
// (RMSNorm gains, LM head, embeddings; Sec. 2.2: they share learning rate and
// weight decay with the Muon-updated matrices).  Adam with bias correction and
// decoupled weight decay:
//   m <- beta1 m + (1-beta1) g;  v <- beta2 v + (1-beta2) g^2
//   p <- p - lr * ( (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps) + wd p )
// One launch covers up to kMaxTensors tensors (their descriptors travel as
// kernel parameters, so nothing is allocated); a pure HBM-streaming kernel:
// 22 bytes per element with bf16 p and g (g 2, m 4+4, v 4+4, p 2+2).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>

#include "../../include/muon.h"

namespace muon {
void set_last_error(const char* msg);
}

namespace {

constexpr int kMaxTensors = 48;
constexpr int kThreads = 128;
constexpr int kCtasPerSm = 16;  // measured best with two 8-element vectors in flight per thread

struct TensorArg {
  void* p;
  const void* g;
  float* m;
  float* v;
  long long numel;
  int p_fp32, g_fp32;
};

struct LaunchArgs {
  TensorArg t[kMaxTensors];
  int count;
  float lr, wd, beta1, beta2, eps;
  float inv_bc1, inv_bc2;  // 1 / (1 - beta^t)
};

__device__ __forceinline__ void load8(const void* base, long long i, bool fp32, float (&out)[8]) {
  if (fp32) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + i));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + i) + 1);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
  } else {
    const uint4 a = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + i));
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      out[2 * e] = __uint_as_float(w[e] << 16);
      out[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
    }
  }
}

__device__ __forceinline__ float adamw_one(float& p, float g, float& m, float& v, const LaunchArgs& A) {
  m = fmaf(A.beta1, m, (1.0f - A.beta1) * g);
  v = fmaf(A.beta2, v, (1.0f - A.beta2) * g * g);
  const float upd = (m * A.inv_bc1) / (sqrtf(v * A.inv_bc2) + A.eps);
  p = p - A.lr * (upd + A.wd * p);
  return p;
}

__global__ void __launch_bounds__(kThreads) adamw_kernel(const __grid_constant__ LaunchArgs A) {
  const TensorArg T = A.t[blockIdx.y];
  const bool vec = ((reinterpret_cast<uintptr_t>(T.p) | reinterpret_cast<uintptr_t>(T.g) |
                     reinterpret_cast<uintptr_t>(T.m) | reinterpret_cast<uintptr_t>(T.v)) & 15) == 0;
  const long long n8 = vec ? T.numel / 8 : 0;
  const long long stride = static_cast<long long>(gridDim.x) * kThreads;
  // two 8-element vectors per thread and trip, all loads issued before the arithmetic
  for (long long i8 = blockIdx.x * static_cast<long long>(kThreads) + threadIdx.x; i8 < n8; i8 += 2 * stride) {
    const long long ia = i8 * 8, ib = (i8 + stride) * 8;
    const bool hb = (i8 + stride) < n8;
    float pa[8], ga[8], ma[8], va[8], pb[8], gb[8], mb[8], vb[8];
    load8(T.g, ia, T.g_fp32 != 0, ga); load8(T.m, ia, true, ma); load8(T.v, ia, true, va); load8(T.p, ia, T.p_fp32 != 0, pa);
    if (hb) { load8(T.g, ib, T.g_fp32 != 0, gb); load8(T.m, ib, true, mb); load8(T.v, ib, true, vb); load8(T.p, ib, T.p_fp32 != 0, pb); }
#pragma unroll
    for (int e = 0; e < 8; ++e) adamw_one(pa[e], ga[e], ma[e], va[e], A);
    if (hb) {
#pragma unroll
      for (int e = 0; e < 8; ++e) adamw_one(pb[e], gb[e], mb[e], vb[e], A);
    }
    for (int h = 0; h < (hb ? 2 : 1); ++h) {
      const long long i = h ? ib : ia;
      float* p = h ? pb : pa; float* m = h ? mb : ma; float* v = h ? vb : va;
      __stcs(reinterpret_cast<float4*>(T.m + i), make_float4(m[0], m[1], m[2], m[3]));
      __stcs(reinterpret_cast<float4*>(T.m + i) + 1, make_float4(m[4], m[5], m[6], m[7]));
      __stcs(reinterpret_cast<float4*>(T.v + i), make_float4(v[0], v[1], v[2], v[3]));
      __stcs(reinterpret_cast<float4*>(T.v + i) + 1, make_float4(v[4], v[5], v[6], v[7]));
      if (T.p_fp32) {
        float* pp = reinterpret_cast<float*>(T.p) + i;
        *reinterpret_cast<float4*>(pp) = make_float4(p[0], p[1], p[2], p[3]);
        *(reinterpret_cast<float4*>(pp) + 1) = make_float4(p[4], p[5], p[6], p[7]);
      } else {
        __nv_bfloat162 hh[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) hh[e] = __floats2bfloat162_rn(p[2 * e], p[2 * e + 1]);
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(T.p) + i) = *reinterpret_cast<const uint4*>(hh);
      }
    }
  }
  // tail (and everything, for tensors that are not 16-byte aligned)
  for (long long i = n8 * 8 + blockIdx.x * static_cast<long long>(kThreads) + threadIdx.x; i < T.numel; i += stride) {
    float g = T.g_fp32 ? reinterpret_cast<const float*>(T.g)[i]
                       : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(T.g)[i]);
    float p = T.p_fp32 ? reinterpret_cast<float*>(T.p)[i] : __bfloat162float(reinterpret_cast<__nv_bfloat16*>(T.p)[i]);
    float m = T.m[i], v = T.v[i];
    adamw_one(p, g, m, v, A);
    T.m[i] = m;
    T.v[i] = v;
    if (T.p_fp32) reinterpret_cast<float*>(T.p)[i] = p;
    else reinterpret_cast<__nv_bfloat16*>(T.p)[i] = __float2bfloat16_rn(p);
  }
}

int fail(int code, const char* msg) {
  muon::set_last_error(msg);
  return code;
}

}  // namespace

extern "C" int muon_adamw_step(const muon_adamw_tensor* tensors, int n_tensors, const muon_adamw_hparams* hp,
                               int device, void* stream_v) {
  if (!tensors || n_tensors <= 0 || !hp) return fail(MUON_ERR_INVALID_ARG, "tensors or hparams is null, or n_tensors <= 0");
  if (hp->step < 1) return fail(MUON_ERR_INVALID_ARG, "step counts from 1");
  if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f && hp->beta2 >= 0.f && hp->beta2 < 1.f) || !(hp->eps >= 0.f) ||
      !std::isfinite(hp->lr) || !std::isfinite(hp->wd))
    return fail(MUON_ERR_INVALID_ARG, "hyper-parameters out of range");
  for (int i = 0; i < n_tensors; ++i) {
    const muon_adamw_tensor& t = tensors[i];
    if (!t.p || !t.g || !t.m || !t.v || t.numel <= 0) return fail(MUON_ERR_INVALID_ARG, "null pointer or non-positive numel");
    if ((t.p_dtype != MUON_DTYPE_BF16 && t.p_dtype != MUON_DTYPE_FP32) ||
        (t.g_dtype != MUON_DTYPE_BF16 && t.g_dtype != MUON_DTYPE_FP32))
      return fail(MUON_ERR_UNSUPPORTED, "dtype must be bf16 or fp32");
    const uintptr_t pa = t.p_dtype == MUON_DTYPE_FP32 ? 3 : 1, ga = t.g_dtype == MUON_DTYPE_FP32 ? 3 : 1;
    if ((reinterpret_cast<uintptr_t>(t.p) & pa) || (reinterpret_cast<uintptr_t>(t.g) & ga) ||
        (reinterpret_cast<uintptr_t>(t.m) & 3) || (reinterpret_cast<uintptr_t>(t.v) & 3))
      return fail(MUON_ERR_ALIGNMENT, "pointer not aligned to its element size");
  }
  cudaError_t ce = cudaSetDevice(device);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, cudaGetErrorString(ce));
  int sms = 0;
  ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, cudaGetErrorString(ce));
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const double bc1 = 1.0 - std::pow(static_cast<double>(hp->beta1), hp->step);
  const double bc2 = 1.0 - std::pow(static_cast<double>(hp->beta2), hp->step);
  for (int first = 0; first < n_tensors; first += kMaxTensors) {
    LaunchArgs A{};
    A.count = n_tensors - first < kMaxTensors ? n_tensors - first : kMaxTensors;
    long long largest = 0;
    for (int i = 0; i < A.count; ++i) {
      const muon_adamw_tensor& t = tensors[first + i];
      A.t[i] = TensorArg{t.p, t.g, t.m, t.v, t.numel, t.p_dtype == MUON_DTYPE_FP32, t.g_dtype == MUON_DTYPE_FP32};
      if (t.numel > largest) largest = t.numel;
    }
    A.lr = hp->lr; A.wd = hp->wd; A.beta1 = hp->beta1; A.beta2 = hp->beta2; A.eps = hp->eps;
    A.inv_bc1 = static_cast<float>(1.0 / bc1);
    A.inv_bc2 = static_cast<float>(1.0 / bc2);
    long long bx = (largest / 8 + kThreads - 1) / kThreads;
    const long long cap = static_cast<long long>(sms) * kCtasPerSm;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    adamw_kernel<<<dim3(static_cast<unsigned>(bx), static_cast<unsigned>(A.count)), kThreads, 0, stream>>>(A);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(MUON_ERR_CUDA, cudaGetErrorString(ce));
  }
  return MUON_OK;
}
