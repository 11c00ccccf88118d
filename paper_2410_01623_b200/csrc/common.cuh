// Shared declarations of the Fira library's translation units: the per-matrix
// device table and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/fira.h"

namespace fira {

// Scalars kept per matrix in the state buffer.  prev_norm and t are optimizer
// state (the "+1" of the paper's comparison table and the step count); the rest
// are diagnostics of the latest step.
struct MatScalars {
  float prev_norm;    // ||S_prev|| after limiting; < 0 means "not set yet"
  float lambda;       // limiter factor of the latest step
  float norm_scaled;  // ||S|| before the limiter
  float k_min, k_max;
  float pad;          // bias factor sqrt(1-b2^s)/(1-b1^s) of the running step (tensor-core path)
  long long t;        // steps taken
};
static_assert(sizeof(MatScalars) == 32, "MatScalars layout");

// One entry of the device-resident problem table.  l = max(m,n) indexes the
// unprojected extent, d = min(m,n) the projected one.
struct MatDev {
  void* W;
  const void* G;
  void* P;            // d x r, row major, dtype
  float* M;           // l x r
  float* V;           // l x r
  MatScalars* sc;
  float* Rt;          // scratch: l x r fp32 low-rank gradient (transposed layout)
  float* Xt;          // scratch: l x r fp32, first N then X = a_low N - a_res lambda k R
  float* kvec;        // scratch: l factors
  float* part;        // scratch: partial sums of ||S||^2
  float* aux;         // scratch: 2 l floats, ||N_l||^2 and ||R_l||^2 (matrix-level factor only)
  __nv_bfloat16* Nb;  // scratch of the tensor-core path: l x r bf16 N
  __nv_bfloat16* Rb;  //   "      l x r bf16 R
  __nv_bfloat16* Xb;  //   "      l x r bf16 X
  float* colpart;     //   "      per (r-tile, l) partial sums of N^2 and R^2, then per-l sums of G^2
  __nv_bfloat16* Gs;  //   "      copies of G and W with 16-byte aligned rows (pitch lds), only when the
  __nv_bfloat16* Ws;  //          caller's rows are not (odd widths): TMA needs aligned rows
  long long lds;
  long long ld;
  int m, n, r;
  int left;           // 1: m <= n (left projection), 0: right projection
  int bf16;           // storage type of W, G, P
  int engine;         // 0 CUDA-core fp32, 1 tcgen05 bf16
  int l, d;
};

struct Hyper {
  float beta1, beta2, eps, lr, a_low, a_res, gamma;
  unsigned mode;      // HYPER_* bits: ablation variants (Section 5.4)
};
enum HyperMode : unsigned {
  HYPER_MATRIX_SCALING = 1u,   // one factor per matrix (Eq. 9)
  HYPER_NO_SCALING = 2u,       // factor 1
  HYPER_NO_RESIDUAL = 4u,      // no residual term (Eq. 6)
  HYPER_PSI_RMSPROP = 8u,      // base optimizer: RMSProp instead of Adam
  HYPER_PSI_ADAGRAD = 16u,     // base optimizer: Adagrad instead of Adam
  HYPER_ONLY_SCALING = 32u,    // Fira-only-scaling: W <- W - lr phi(R) G (no P N term, S = G diag k)
};

enum DeviceStatusBits : unsigned {
  DEV_STATUS_TIMEOUT = 1u,
  DEV_STATUS_NONFINITE = 2u,
};

template <typename T>
__device__ __forceinline__ float to_float(T v);
template <>
__device__ __forceinline__ float to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}
template <typename T>
__device__ __forceinline__ T from_float(float v);
template <>
__device__ __forceinline__ float from_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

// Index of the matrix whose tile range contains `tile`: the largest i with
// start[i] <= tile (start has count + 1 ascending entries).
__device__ __forceinline__ int find_matrix(const int* __restrict__ start, int count, int tile) {
  int lo = 0, hi = count;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (start[mid] <= tile) lo = mid; else hi = mid;
  }
  return lo;
}

void set_error(const std::string& msg);

// Optional per-kernel timing of a step: marks are CUDA events recorded between the
// launches.  slot = the step's row of the event ring, next = the next mark.
struct PhaseTimer {
  bool on = false;
  std::vector<cudaEvent_t> events;   // FIRA_TIMING_MAX_STEPS x (FIRA_TIMING_MAX_PHASES + 1)
  std::vector<const char*> names;    // phase names in launch order
  int slot = 0, next = 0;
  long long steps = 0;               // steps recorded since enabling
  void begin_step() { next = 0; slot = (int)(steps % FIRA_TIMING_MAX_STEPS); }
  void mark(cudaStream_t st) {
    if (!on || next > FIRA_TIMING_MAX_PHASES) return;
    cudaEventRecord(events[(size_t)slot * (FIRA_TIMING_MAX_PHASES + 1) + next], st);
    ++next;
  }
};

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

}  // namespace fira
