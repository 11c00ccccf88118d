// Plain Adam (Eq. 1-4) for the parameters that are not projected: embeddings, the output head,
// norm gains.  One grouped, HBM-bound kernel over a list of flat tensors; the pointer table
// travels in the kernel arguments, so nothing is allocated.
//
//   M <- b1 M + (1-b1) G;  V <- b2 V + (1-b2) G^2;
//   W <- W - lr sqrt(1-b2^s)/(1-b1^s) M / (sqrt V + eps),  s = t + 1
//
// Bytes per element: G and W read, W written (3 e) plus M and V read and written (16).
#include <math.h>

#include <algorithm>

#include "common.cuh"
#include "context.cuh"

namespace fira {
namespace {

constexpr int AD_TENSORS = 24;            // tensors per launch
constexpr int AD_THREADS = 256;
constexpr int AD_PER_THREAD = 16;         // elements per thread (4 vectors of 4)
constexpr int AD_BLOCK_ELEMS = AD_THREADS * AD_PER_THREAD;

struct AdamChunk {
  void* W[AD_TENSORS];
  const void* G[AD_TENSORS];
  float* M[AD_TENSORS];
  float* V[AD_TENSORS];
  long long numel[AD_TENSORS];
  int block_start[AD_TENSORS + 1];
  int count;
};

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
  const float4 u = *reinterpret_cast<const float4*>(p);
  v[0] = u.x; v[1] = u.y; v[2] = u.z; v[3] = u.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(u.x << 16); v[1] = __uint_as_float(u.x & 0xffff0000u);
  v[2] = __uint_as_float(u.y << 16); v[3] = __uint_as_float(u.y & 0xffff0000u);
}
__device__ __forceinline__ void store4(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&v)[4]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  uint2 u;
  u.x = *reinterpret_cast<unsigned*>(&a); u.y = *reinterpret_cast<unsigned*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

template <typename T>
__global__ void __launch_bounds__(AD_THREADS)
k_adam_dense(const __grid_constant__ AdamChunk ch, float beta1, float beta2, float eps, float step) {
  int q = 0;
  while (q + 1 < ch.count && (int)blockIdx.x >= ch.block_start[q + 1]) ++q;
  T* W = static_cast<T*>(ch.W[q]);
  const T* G = static_cast<const T*>(ch.G[q]);
  float* M = ch.M[q];
  float* V = ch.V[q];
  const long long n = ch.numel[q];
  const long long base = (long long)(blockIdx.x - ch.block_start[q]) * AD_BLOCK_ELEMS;
#pragma unroll
  for (int u = 0; u < AD_PER_THREAD / 4; ++u) {
    const long long i = base + ((long long)u * AD_THREADS + threadIdx.x) * 4;
    if (i + 4 <= n) {
      float g[4], w[4], m[4], v[4];
      load4<T>(G + i, g);
      load4<T>(W + i, w);
      load4<float>(M + i, m);
      load4<float>(V + i, v);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        m[e] = beta1 * m[e] + (1.f - beta1) * g[e];
        v[e] = beta2 * v[e] + (1.f - beta2) * g[e] * g[e];
        w[e] = w[e] - step * m[e] / (sqrtf(v[e]) + eps);
      }
      store4(M + i, m);
      store4(V + i, v);
      store4(W + i, w);
    } else {
      for (long long j = i; j < n; ++j) {
        const float g = to_float<T>(G[j]);
        const float m = beta1 * M[j] + (1.f - beta1) * g;
        const float v = beta2 * V[j] + (1.f - beta2) * g * g;
        M[j] = m; V[j] = v;
        W[j] = from_float<T>(to_float<T>(W[j]) - step * m / (sqrtf(v) + eps));
      }
    }
  }
}

}  // namespace
}  // namespace fira

using namespace fira;

extern "C" fira_status fira_adam_dense(const fira_hparams* hp, int32_t count, void* const* W_dev,
                                       const void* const* G_dev, float* const* M_dev, float* const* V_dev,
                                       const int64_t* numel, fira_dtype dtype, int64_t t, float lr,
                                       void* cuda_stream) {
  if (!hp || count <= 0 || !W_dev || !G_dev || !M_dev || !V_dev || !numel) {
    set_error("fira_adam_dense: null argument or empty list"); return FIRA_ERR_INVALID_ARG;
  }
  if (!(hp->eps > 0.f) || !(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f) || t < 0) {
    set_error("fira_adam_dense: need eps > 0, beta1 and beta2 in [0, 1), t >= 0"); return FIRA_ERR_INVALID_ARG;
  }
  if (dtype != FIRA_F32 && dtype != FIRA_BF16) { set_error("unknown dtype"); return FIRA_ERR_INVALID_ARG; }
  if (!(lr < 0.f) && !isfinite(lr)) { set_error("lr must be finite"); return FIRA_ERR_INVALID_ARG; }
  for (int i = 0; i < count; ++i) {
    if (!W_dev[i] || !G_dev[i] || !M_dev[i] || !V_dev[i] || numel[i] <= 0 ||
        (((uintptr_t)W_dev[i] | (uintptr_t)G_dev[i] | (uintptr_t)M_dev[i] | (uintptr_t)V_dev[i]) & 15)) {
      set_error("fira_adam_dense: tensor " + std::to_string(i) + ": pointers must be non-null and 16-byte aligned, numel > 0");
      return FIRA_ERR_INVALID_ARG;
    }
    if ((numel[i] + AD_BLOCK_ELEMS - 1) / AD_BLOCK_ELEMS > (1ll << 30)) { set_error("tensor too large"); return FIRA_ERR_INVALID_ARG; }
  }
  // every chunk's block count is checked before the first launch: an error leaves all tensors untouched
  for (int first = 0; first < count; first += AD_TENSORS) {
    long long blocks = 0;
    for (int q = 0; q < std::min(AD_TENSORS, count - first); ++q)
      blocks += (numel[first + q] + AD_BLOCK_ELEMS - 1) / AD_BLOCK_ELEMS;
    if (blocks > 0x7fffffffll) { set_error("fira_adam_dense: too many elements in one call"); return FIRA_ERR_INVALID_ARG; }
  }
  const double s = (double)(t + 1);
  const float bias = (float)(sqrt(1.0 - pow((double)hp->beta2, s)) / (1.0 - pow((double)hp->beta1, s)));
  const float step = (lr < 0.f ? hp->lr : lr) * bias;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  for (int first = 0; first < count; first += AD_TENSORS) {
    AdamChunk ch;
    ch.count = std::min(AD_TENSORS, count - first);
    long long blocks = 0;
    for (int q = 0; q < ch.count; ++q) {
      ch.W[q] = W_dev[first + q]; ch.G[q] = G_dev[first + q]; ch.M[q] = M_dev[first + q]; ch.V[q] = V_dev[first + q];
      ch.numel[q] = numel[first + q];
      ch.block_start[q] = (int)blocks;
      blocks += (numel[first + q] + AD_BLOCK_ELEMS - 1) / AD_BLOCK_ELEMS;
    }
    ch.block_start[ch.count] = (int)blocks;
    if (dtype == FIRA_BF16)
      k_adam_dense<__nv_bfloat16><<<(unsigned)blocks, AD_THREADS, 0, st>>>(ch, hp->beta1, hp->beta2, hp->eps, step);
    else
      k_adam_dense<float><<<(unsigned)blocks, AD_THREADS, 0, st>>>(ch, hp->beta1, hp->beta2, hp->eps, step);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_error(std::string("fira_adam_dense: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  return FIRA_OK;
}
