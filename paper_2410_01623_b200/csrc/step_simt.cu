// fp32 CUDA-core kernels of the Fira step (Algorithm 1's loop body), grouped over
// a list of matrices: one launch per phase covers every matrix of the list.
//
// Phases (l = unprojected index, d = projected index, Pi = the d x r projection):
//   1. project      Rt[l][j]   = sum_d G(d,l) Pi[d][j]                      (R = P^T G)
//   2. adam_rows    M,V update, N, k_l = ||N_l|| / (||R_l|| + eps)           (Eq. 2-4, Eq. 11)
//   3. back_project mode NORM:   part = sum (k_l (G - Pi R))^2               (||S||, literal residual)
//   4. finalize     lambda, ||S_prev||, t                                    (Eq. 12)
//   5. form_x       Xt = a_low N - a_res lambda k_l R
//   6. back_project mode UPDATE: W -= lr (Pi X + a_res lambda k_l G)
// Phase 6 uses the identity alpha (P N + lambda (G - P R) diag k) =
// P (alpha N - alpha lambda R diag k) + alpha lambda G diag k, so that the update
// needs one product instead of two.
#include "common.cuh"
#include "simt_gemm.cuh"
#include "step_simt.cuh"

namespace fira {

namespace {

__device__ __forceinline__ int simt_tiles_dev(int extent) { return (extent + SIMT_TILE - 1) / SIMT_TILE; }

// ---------------------------------------------------------------- phase 1
template <typename T>
__device__ __forceinline__ void project_tile(const MatDev& mt, int tile, float (*As)[SIMT_TILE + 4],
                                             float (*Bs)[SIMT_TILE + 4]) {
  const int rt = simt_tiles_dev(mt.r);
  const int i0 = (tile / rt) * SIMT_TILE, j0 = (tile % rt) * SIMT_TILE;
  float acc[4 * SIMT_Q][4 * SIMT_Q] = {};
  const T* G = static_cast<const T*>(mt.G);
  const T* P = static_cast<const T*>(mt.P);
  // A(i = l, k = d): G[d][l] when left, G[l][d] when right.
  const long long sAi = mt.left ? 1 : mt.ld, sAk = mt.left ? mt.ld : 1;
  gemm_tile<SIMT_Q, T, T>(G, sAi, sAk, P, mt.r, 1, mt.l, mt.r, mt.d, i0, j0, acc, As, Bs);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int x = 0; x < 4 * SIMT_Q; ++x) {
    const int i = i0 + tile_coord(ty, x);
    if (i >= mt.l) continue;
#pragma unroll
    for (int y = 0; y < 4 * SIMT_Q; ++y) {
      const int j = j0 + tile_coord(tx, y);
      if (j < mt.r) mt.Rt[(long long)i * mt.r + j] = acc[x][y];
    }
  }
}

__global__ void __launch_bounds__(GEMM_THREADS, 2)
k_project(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
          const int* __restrict__ tile_start, int first) {
  __shared__ __align__(16) float As[TK][SIMT_TILE + 4];
  __shared__ __align__(16) float Bs[TK][SIMT_TILE + 4];
  const int gt = blockIdx.x + first;
  const int p = find_matrix(tile_start, nlist, gt);
  const MatDev mt = mats[list[p]];
  const int tile = gt - tile_start[p];
  if (mt.bf16) project_tile<__nv_bfloat16>(mt, tile, As, Bs);
  else project_tile<float>(mt, tile, As, Bs);
}

// ---------------------------------------------------------------- phase 2
// One warp per unprojected index l.  N goes to Xt.
__global__ void __launch_bounds__(256)
k_adam_rows(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
            const int* __restrict__ row_start, int first_row, int rows_total, Hyper hp) {
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int row = first_row + blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  if (row >= rows_total) return;
  const int p = find_matrix(row_start, nlist, row);
  const MatDev mt = mats[list[p]];
  const int l = row - row_start[p];
  // bias correction sqrt(1 - b2^s) / (1 - b1^s), s = t + 1, in double
  const double s = (double)(mt.sc->t + 1);
  const float bias = (float)(sqrt(1.0 - pow((double)hp.beta2, s)) / (1.0 - pow((double)hp.beta1, s)));
  const long long base = (long long)l * mt.r;
  float nn = 0.f, rn = 0.f;
  // four entries per lane at a time, their loads before their stores (see back_tile)
  for (int jq = lane; jq < mt.r; jq += 128) {
    float rv4[4], m4[4], v4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = jq + 32 * u;
      const bool in = j < mt.r;
      rv4[u] = in ? mt.Rt[base + j] : 0.f;
      v4[u] = in ? mt.V[base + j] : 0.f;
      m4[u] = (in && !(hp.mode & (HYPER_PSI_RMSPROP | HYPER_PSI_ADAGRAD))) ? mt.M[base + j] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = jq + 32 * u;
      if (j >= mt.r) continue;
      const float rv = rv4[u];
      float vv, nv;
      if (hp.mode & HYPER_PSI_RMSPROP) {
        vv = hp.beta2 * v4[u] + (1.f - hp.beta2) * rv * rv;
        nv = rv / (sqrtf(vv) + hp.eps);
      } else if (hp.mode & HYPER_PSI_ADAGRAD) {
        vv = v4[u] + rv * rv;
        nv = rv / (sqrtf(vv) + hp.eps);
      } else {
        const float mv = hp.beta1 * m4[u] + (1.f - hp.beta1) * rv;
        vv = hp.beta2 * v4[u] + (1.f - hp.beta2) * rv * rv;
        mt.M[base + j] = mv;
        nv = bias * mv / (sqrtf(vv) + hp.eps);
      }
      mt.V[base + j] = vv;
      mt.Xt[base + j] = nv;
      nn = fmaf(nv, nv, nn);
      rn = fmaf(rv, rv, rn);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    nn += __shfl_xor_sync(0xffffffffu, nn, o);
    rn += __shfl_xor_sync(0xffffffffu, rn, o);
  }
  if (lane == 0) {
    if (hp.mode & HYPER_MATRIX_SCALING) {        // the factor comes from the whole matrix: k_finalize
      mt.aux[l] = nn; mt.aux[mt.l + l] = rn; mt.kvec[l] = 1.f;
    } else if (hp.mode & HYPER_NO_SCALING) {
      mt.kvec[l] = 1.f;
    } else {
      mt.kvec[l] = sqrtf(nn) / (sqrtf(rn) + hp.eps);
    }
  }
}

// ---------------------------------------------------------------- phases 3 and 6
enum { MODE_NORM = 0, MODE_UPDATE = 1 };

template <typename T, int MODE>
__device__ __forceinline__ void back_tile(const MatDev& mt, int tile, float lr, float a_res,
                                          float (*As)[SIMT_TILE + 4], float (*Bs)[SIMT_TILE + 4], float* red) {
  const int ct = simt_tiles_dev(mt.n);
  const int i0 = (tile / ct) * SIMT_TILE, j0 = (tile % ct) * SIMT_TILE;
  float acc[4 * SIMT_Q][4 * SIMT_Q] = {};
  const T* P = static_cast<const T*>(mt.P);
  const float* X = (MODE == MODE_NORM) ? mt.Rt : mt.Xt;
  const long long r = mt.r;
  if (mt.left) {
    // D[d][l] = sum_j Pi[d][j] X[l][j]
    gemm_tile<SIMT_Q, T, float>(P, r, 1, X, 1, r, mt.m, mt.n, mt.r, i0, j0, acc, As, Bs);
  } else {
    // D[l][d] = sum_j X[l][j] Pi[d][j]
    gemm_tile<SIMT_Q, float, T>(X, r, 1, P, 1, r, mt.m, mt.n, mt.r, i0, j0, acc, As, Bs);
  }
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const T* G = static_cast<const T*>(mt.G);
  T* W = static_cast<T*>(mt.W);
  const float lam = (MODE == MODE_UPDATE) ? mt.sc->lambda : 1.f;
  float ss = 0.f;
  // Two rows of the thread's entries at a time: every load of the pair first, then the arithmetic
  // and the stores.  (Written element by element, each load of G and W would wait for the store
  // before it, since the compiler cannot tell that they never overlap.)
#pragma unroll
  for (int xb = 0; xb < 4 * SIMT_Q; xb += 2) {
    float g[2][4 * SIMT_Q], w[2][4 * SIMT_Q], kf[2][4 * SIMT_Q];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      const int i = i0 + tile_coord(ty, xb + x);
#pragma unroll
      for (int y = 0; y < 4 * SIMT_Q; ++y) {
        const int j = j0 + tile_coord(tx, y);
        const bool in = i < mt.m && j < mt.n;
        const long long off = (long long)i * mt.ld + j;
        kf[x][y] = in ? mt.kvec[mt.left ? j : i] : 0.f;
        g[x][y] = in ? to_float<T>(G[off]) : 0.f;
        w[x][y] = (MODE == MODE_UPDATE && in) ? to_float<T>(W[off]) : 0.f;
      }
    }
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      const int i = i0 + tile_coord(ty, xb + x);
      if (i >= mt.m) continue;
#pragma unroll
      for (int y = 0; y < 4 * SIMT_Q; ++y) {
        const int j = j0 + tile_coord(tx, y);
        if (j >= mt.n) continue;
        if (MODE == MODE_NORM) {
          const float sv = kf[x][y] * (g[x][y] - acc[xb + x][y]);
          ss = fmaf(sv, sv, ss);
        } else {
          W[(long long)i * mt.ld + j] =
              from_float<T>(w[x][y] - lr * (acc[xb + x][y] + a_res * lam * kf[x][y] * g[x][y]));
        }
      }
    }
  }
  if (MODE == MODE_NORM) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int w = 0; w < GEMM_THREADS / 32; ++w) tot += red[w];
      mt.part[tile] = tot;
    }
  }
}

template <int MODE>
__global__ void __launch_bounds__(GEMM_THREADS, 2)
k_back_project(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
               const int* __restrict__ tile_start, int first, float lr, float a_res) {
  __shared__ __align__(16) float As[TK][SIMT_TILE + 4];
  __shared__ __align__(16) float Bs[TK][SIMT_TILE + 4];
  __shared__ float red[GEMM_THREADS / 32];
  const int gt = blockIdx.x + first;
  const int p = find_matrix(tile_start, nlist, gt);
  const MatDev mt = mats[list[p]];
  const int tile = gt - tile_start[p];
  if (mt.bf16) back_tile<__nv_bfloat16, MODE>(mt, tile, lr, a_res, As, Bs, red);
  else back_tile<float, MODE>(mt, tile, lr, a_res, As, Bs, red);
}

// ---------------------------------------------------------------- phase 5
__global__ void __launch_bounds__(256)
k_form_x(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
         const int* __restrict__ row_start, int first_row, int rows_total, float a_low, float a_res) {
  const int lane = threadIdx.x & 31;
  const int row = first_row + blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows_total) return;
  const int p = find_matrix(row_start, nlist, row);
  const MatDev mt = mats[list[p]];
  const int l = row - row_start[p];
  const float c = a_res * mt.sc->lambda * mt.kvec[l];
  const long long base = (long long)l * mt.r;
  for (int jq = lane; jq < mt.r; jq += 128) {    // four entries per lane, loads before stores
    float n4[4], r4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = jq + 32 * u;
      n4[u] = j < mt.r ? mt.Xt[base + j] : 0.f;
      r4[u] = j < mt.r ? mt.Rt[base + j] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = jq + 32 * u;
      if (j < mt.r) mt.Xt[base + j] = a_low * n4[u] - c * r4[u];
    }
  }
}

// ---------------------------------------------------------------- Fira-only-scaling
// W <- W - lr phi(R) G: no product.  One block per tile x tile block of W; rows are walked by the
// warps, columns by the lanes (coalesced along the rows of G and W).
template <typename T, int UPDATE>
__device__ __forceinline__ float scaled_gradient_tile(const MatDev& mt, int i0, int j0, int tile, float c) {
  const T* G = static_cast<const T*>(mt.G);
  T* W = static_cast<T*>(mt.W);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int i1 = min(i0 + tile, mt.m), j1 = min(j0 + tile, mt.n);
  float ss = 0.f;
  for (int i = i0 + warp; i < i1; i += 8) {
    const float krow = mt.left ? 0.f : mt.kvec[i];
    for (int j = j0 + lane; j < j1; j += 32) {
      const float kf = mt.left ? mt.kvec[j] : krow;
      const long long off = (long long)i * mt.ld + j;
      const float g = to_float<T>(G[off]);
      if (UPDATE) W[off] = from_float<T>(to_float<T>(W[off]) - c * kf * g);
      else { const float sv = kf * g; ss = fmaf(sv, sv, ss); }
    }
  }
  return ss;
}

template <int UPDATE>
__global__ void __launch_bounds__(256)
k_scaled_gradient(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
                  const int* __restrict__ tile_start, int first, int tile, float lr, float a_res) {
  __shared__ float red[8];
  const int gt = blockIdx.x + first;
  const int p = find_matrix(tile_start, nlist, gt);
  const MatDev mt = mats[list[p]];
  const int t = gt - tile_start[p];
  const int ct = (mt.n + tile - 1) / tile;
  const int i0 = (t / ct) * tile, j0 = (t % ct) * tile;
  const float c = UPDATE ? lr * a_res * mt.sc->lambda : 0.f;
  float ss = mt.bf16 ? scaled_gradient_tile<__nv_bfloat16, UPDATE>(mt, i0, j0, tile, c)
                     : scaled_gradient_tile<float, UPDATE>(mt, i0, j0, tile, c);
  if (!UPDATE) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int w = 0; w < 8; ++w) tot += red[w];
      mt.part[t] = tot;
    }
  }
}

}  // namespace

void launch_scaled_gradient(const MatDev* mats, const int* list, int nlist, const int* tile_start, int first,
                            int tiles, int tile, int update, float lr, float a_res, cudaStream_t st) {
  if (tiles <= 0) return;
  if (update) k_scaled_gradient<1><<<tiles, 256, 0, st>>>(mats, list, nlist, tile_start, first, tile, lr, a_res);
  else k_scaled_gradient<0><<<tiles, 256, 0, st>>>(mats, list, nlist, tile_start, first, tile, lr, a_res);
}

// ---------------------------------------------------------------- phase 4
__global__ void __launch_bounds__(256)
k_finalize(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
           const int* __restrict__ npart_of, Hyper hp, unsigned* __restrict__ status) {
  __shared__ double sred[256];
  __shared__ float smin[256], smax[256];
  const MatDev mt = mats[list[blockIdx.x]];
  const int npart = npart_of[blockIdx.x];
  double acc = 0.0;
  for (int i = threadIdx.x; i < npart; i += 256) acc += (double)mt.part[i];
  // Matrix-level factor (Eq. 9): the phases before ran with k = 1, so `part` holds ||G - P R||^2;
  // the factor scales the norm here and fills the k table for the phases after.
  float kmat = 1.f;
  if (hp.mode & HYPER_MATRIX_SCALING) {
    __shared__ double sn[256], sr[256];
    double an = 0.0, ar = 0.0;
    for (int i = threadIdx.x; i < mt.l; i += 256) { an += (double)mt.aux[i]; ar += (double)mt.aux[mt.l + i]; }
    sn[threadIdx.x] = an; sr[threadIdx.x] = ar;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
      if (threadIdx.x < o) { sn[threadIdx.x] += sn[threadIdx.x + o]; sr[threadIdx.x] += sr[threadIdx.x + o]; }
      __syncthreads();
    }
    kmat = (float)(sqrt(sn[0]) / (sqrt(sr[0]) + (double)hp.eps));
    for (int i = threadIdx.x; i < mt.l; i += 256) mt.kvec[i] = kmat;
  }
  float kmin = INFINITY, kmax = -INFINITY;
  for (int i = threadIdx.x; i < mt.l; i += 256) {
    const float kv = (hp.mode & HYPER_MATRIX_SCALING) ? kmat : mt.kvec[i];
    kmin = fminf(kmin, kv);
    kmax = fmaxf(kmax, kv);
  }
  sred[threadIdx.x] = acc; smin[threadIdx.x] = kmin; smax[threadIdx.x] = kmax;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sred[threadIdx.x] += sred[threadIdx.x + o];
      smin[threadIdx.x] = fminf(smin[threadIdx.x], smin[threadIdx.x + o]);
      smax[threadIdx.x] = fmaxf(smax[threadIdx.x], smax[threadIdx.x + o]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double tot = sred[0] > 0.0 ? sred[0] : 0.0;
    const float norm = kmat * (float)sqrt(tot);
    const float prev = mt.sc->prev_norm;
    float lam = 1.f;
    if (hp.mode & HYPER_NO_RESIDUAL) {           // Eq. 6: no residual, nothing to limit or remember
      mt.sc->norm_scaled = 0.f;
      mt.sc->lambda = 1.f;
      mt.sc->k_min = 0.f;
      mt.sc->k_max = 0.f;
      mt.sc->t = mt.sc->t + 1;
      return;
    }
    if (prev >= 0.f && !isinf(hp.gamma)) {
      const float ratio = norm / (prev + hp.eps);
      lam = hp.gamma / fmaxf(ratio, hp.gamma);
    }
    if (!isfinite((float)sred[0]) || !isfinite(smax[0])) atomicOr(status, DEV_STATUS_NONFINITE);
    mt.sc->norm_scaled = norm;
    mt.sc->lambda = lam;
    mt.sc->prev_norm = lam * norm;
    mt.sc->k_min = smin[0];
    mt.sc->k_max = smax[0];
    mt.sc->t = mt.sc->t + 1;
  }
}

const char* const kSimtPhaseNames[6] = {"k_project", "k_adam_rows", "k_back_project<norm>",
                                        "k_finalize", "k_form_x", "k_back_project<update>"};

int launch_simt_step(const SimtPlan& pl, const Hyper& hp, unsigned* status_dev, cudaStream_t st,
                     PhaseTimer* tm, int qa, int qb) {
  if (pl.nlist == 0) return 0;
  // the sub-range [qa, qb) of the list: first tile / row and their counts from the host copies of
  // the prefix arrays; the kernels still search the whole arrays with absolute indices
  int pt0 = 0, pt1 = pl.proj_tiles, r0 = 0, r1 = pl.rows_total, wt0 = 0, wt1 = pl.w_tiles, nq = pl.nlist;
  if (qb >= 0) {
    if (qa >= qb) return 0;
    pt0 = pl.h_proj_tile_start[qa]; pt1 = pl.h_proj_tile_start[qb];
    r0 = pl.h_row_start[qa]; r1 = pl.h_row_start[qb];
    wt0 = pl.h_w_tile_start[qa]; wt1 = pl.h_w_tile_start[qb];
    nq = qb - qa;
  } else {
    qa = 0;
  }
  tm->mark(st);
  k_project<<<pt1 - pt0, GEMM_THREADS, 0, st>>>(pl.mats, pl.list, pl.nlist, pl.proj_tile_start, pt0);
  tm->mark(st);
  const int row_blocks = (r1 - r0 + 7) / 8;
  k_adam_rows<<<row_blocks, 256, 0, st>>>(pl.mats, pl.list, pl.nlist, pl.row_start, r0, r1, hp);
  tm->mark(st);
  if (hp.mode & HYPER_ONLY_SCALING) {
    // W <- W - lr phi(R) G: the norm of the scaled gradient, the limiter, the element-wise update
    launch_scaled_gradient(pl.mats, pl.list, pl.nlist, pl.w_tile_start, wt0, wt1 - wt0, SIMT_TILE, 0, 0.f, hp.a_res, st);
    tm->mark(st);
    k_finalize<<<nq, 256, 0, st>>>(pl.mats, pl.list + qa, nq, pl.npart + qa, hp, status_dev);
    tm->mark(st);
    tm->mark(st);
    launch_scaled_gradient(pl.mats, pl.list, pl.nlist, pl.w_tile_start, wt0, wt1 - wt0, SIMT_TILE, 1, hp.lr, hp.a_res, st);
    tm->mark(st);
    return 5;
  }
  k_back_project<MODE_NORM><<<wt1 - wt0, GEMM_THREADS, 0, st>>>(pl.mats, pl.list, pl.nlist,
                                                                pl.w_tile_start, wt0, 0.f, hp.a_res);
  tm->mark(st);
  k_finalize<<<nq, 256, 0, st>>>(pl.mats, pl.list + qa, nq, pl.npart + qa, hp, status_dev);
  tm->mark(st);
  k_form_x<<<row_blocks, 256, 0, st>>>(pl.mats, pl.list, pl.nlist, pl.row_start, r0, r1, hp.a_low, hp.a_res);
  tm->mark(st);
  k_back_project<MODE_UPDATE><<<wt1 - wt0, GEMM_THREADS, 0, st>>>(pl.mats, pl.list, pl.nlist,
                                                                  pl.w_tile_start, wt0, hp.lr, hp.a_res);
  tm->mark(st);
  return 6;
}

}  // namespace fira
