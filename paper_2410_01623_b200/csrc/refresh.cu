// Projection refresh (Eq. 7): an orthonormal basis of the dominant rank-r singular
// subspace of G, by blocked subspace iteration on the device.
//
// With A = G seen as a d x l matrix (d = projected extent):
//   Z <- Gaussian (l x r);  Y <- orth(A Z)
//   repeat `iters` times:   Z <- orth(A^T Y);  Y <- orth(A Z)
//   projection <- Y  (d x r)
// orth() is CholeskyQR: C = Y^T Y, C = L L^T, Y <- Y L^-T, once for the intermediate
// iterates and twice for the basis that is kept.  It changes the basis, never the
// spanned subspace, so a small diagonal shift in the first pass (which keeps the
// factorisation defined for ill-conditioned Y) costs no accuracy of the subspace.
// The paper calls a library SVD here; the iteration converges to the same subspace
// at the rate (sigma_{r+1}/sigma_r)^2 per round.
//
// Everything runs on the CUDA cores in fp32, except for bf16 matrices of tensor-core size with
// TMA-readable rows.  For those every product of the iteration is a job of the step's projection
// kernel in its plain-output mode (fp32 accumulation in tensor memory):
//   * A Z and A^T Y: G is exact in bf16; the iterate is rounded to bf16, and in the last round it is
//     split into a bf16 high part and a bf16 remainder (two k-segments), so that the basis that is
//     kept carries no bf16 rounding of the iterate;
//   * the Gram product Y^T Y and the application of the inverse factor Y <- Y L^-T: for the basis
//     that is kept both operands are fp32 matrices split into two bf16 parts, three k-segments
//     (hi hi + hi lo + lo hi), which is good to about 2^-16: enough for CholeskyQR, whose second pass
//     removes what the first left; for the intermediate iterates plain bf16 operands (one segment):
//     the next product rounds the iterate to bf16 anyway, and all it asks is a well-conditioned one;
//   * L^-T itself comes from the triangular-solve kernel applied to the identity (r x r, fp32).
// Only the Cholesky factorisation and that small solve stay on the CUDA cores.
//
// Random numbers: Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy
// as 1, 2, 3", SC'11), keyed by the caller's seed, turned into normals by the
// Box-Muller transform.
#include <algorithm>

#include "context.cuh"
#include "simt_gemm.cuh"
#include "step_tc.cuh"

namespace fira {

namespace {

struct RefreshMat {
  const void* G;
  void* P;
  float* Y;   // d x r
  float* Z;   // l x r
  float* C;   // r x r
  float* U;            // r x r: L^-T (tc only)
  __nv_bfloat16* Yb;   // bf16 high parts of Y, Z, U: operands of the tensor-core products (tc only)
  __nv_bfloat16* Zb;
  __nv_bfloat16* Ub;
  __nv_bfloat16* Yl;   // bf16 remainders: X - bf16(X)
  __nv_bfloat16* Zl;
  __nv_bfloat16* Ul;
  float* out32;        // optional copy of the kept basis in fp32, before it is rounded for storage
  float* info;         // a few floats of the Cholesky factorisation (pivot floor)
  int tc;              // every product of this matrix runs on the tensor cores
  long long ld;
  int d, l, r;
  int left, bf16;
  unsigned long long key;
};

struct GemmDesc {
  const void* A; long long sAi, sAk; int a_bf16;
  const float* B; long long sBk, sBj;
  float* C; long long sCi;
  int I, J, K;
};

// ------------------------------------------------------------------ Philox4x32-10
__device__ __forceinline__ void philox4x32_10(unsigned c0, unsigned c1, unsigned c2, unsigned c3,
                                              unsigned k0, unsigned k1, unsigned (&out)[4]) {
  const unsigned M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const unsigned hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const unsigned hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const unsigned n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__global__ void __launch_bounds__(256)
k_gauss(const RefreshMat* __restrict__ rm) {
  const RefreshMat m = rm[blockIdx.y];
  const long long total = (long long)m.l * m.r;
  const long long quads = (total + 3) / 4;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < quads;
       q += (long long)gridDim.x * blockDim.x) {
    unsigned o[4];
    philox4x32_10((unsigned)q, (unsigned)(q >> 32), 0u, 0u, (unsigned)m.key, (unsigned)(m.key >> 32), o);
    // two Box-Muller pairs; the radius uniforms lie in (0, 1]
    const float u0 = ((float)(o[0] >> 8) + 1.0f) * (1.0f / 16777216.0f);
    const float u1 = (float)(o[1] >> 8) * (1.0f / 16777216.0f);
    const float u2 = ((float)(o[2] >> 8) + 1.0f) * (1.0f / 16777216.0f);
    const float u3 = (float)(o[3] >> 8) * (1.0f / 16777216.0f);
    const float ra = sqrtf(-2.0f * logf(u0)), rb = sqrtf(-2.0f * logf(u2));
    float s0, c0, s1, c1;
    sincospif(2.0f * u1, &s0, &c0);
    sincospif(2.0f * u3, &s1, &c1);
    const float v[4] = {ra * c0, ra * s0, rb * c1, rb * s1};
    for (int e = 0; e < 4; ++e) {
      const long long idx = q * 4 + e;
      if (idx < total) m.Z[idx] = v[e];
    }
  }
}

// ------------------------------------------------------------------ grouped product
__global__ void __launch_bounds__(GEMM_THREADS, 2)
k_rgemm(const GemmDesc* __restrict__ descs, int ndesc, const int* __restrict__ tile_start) {
  __shared__ __align__(16) float As[TK][SIMT_TILE + 4];
  __shared__ __align__(16) float Bs[TK][SIMT_TILE + 4];
  const int p = find_matrix(tile_start, ndesc, blockIdx.x);
  const GemmDesc g = descs[p];
  const int tile = blockIdx.x - tile_start[p];
  const int jt = (g.J + SIMT_TILE - 1) / SIMT_TILE;
  const int i0 = (tile / jt) * SIMT_TILE, j0 = (tile % jt) * SIMT_TILE;
  float acc[4 * SIMT_Q][4 * SIMT_Q] = {};
  if (g.a_bf16)
    gemm_tile<SIMT_Q, __nv_bfloat16, float>((const __nv_bfloat16*)g.A, g.sAi, g.sAk, g.B, g.sBk, g.sBj,
                                    g.I, g.J, g.K, i0, j0, acc, As, Bs);
  else
    gemm_tile<SIMT_Q, float, float>((const float*)g.A, g.sAi, g.sAk, g.B, g.sBk, g.sBj, g.I, g.J, g.K,
                            i0, j0, acc, As, Bs);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int x = 0; x < 4 * SIMT_Q; ++x) {
    const int i = i0 + tile_coord(ty, x);
    if (i >= g.I) continue;
#pragma unroll
    for (int y = 0; y < 4 * SIMT_Q; ++y) {
      const int j = j0 + tile_coord(tx, y);
      if (j < g.J) g.C[(long long)i * g.sCi + j] = acc[x][y];
    }
  }
}

// ------------------------------------------------------------------ Cholesky
// C (r x r, symmetric, row major) -> lower factor L in place (the strict upper triangle is left as
// it was), for all matrices of a chunk at once, right-looking over block columns of CB = 64.  Three
// launches per block column, each over every matrix:
//   k_chol_diag   one block per matrix factors the CB x CB diagonal block, one row per thread in registers
//   k_chol_panel  the rows below it: L[i, J] = C[i, J] L_JJ^-T, 64 rows per block
//   k_chol_update the trailing matrix: C[I, K] -= L[I, J] L[K, J]^T on 128 x 128 tiles of its lower half
// On the first block column k_chol_diag also adds shift_rel * trace(C)/r to the whole diagonal and
// notes the pivot floor in info[0].  A non-positive or non-finite pivot is replaced and flagged.
// Matrices whose r does not reach the block column do nothing.
constexpr int CB = 64;

__global__ void __launch_bounds__(GEMM_THREADS)
k_chol_diag(const RefreshMat* __restrict__ rm, int J0, float shift_rel, unsigned* __restrict__ status) {
  __shared__ float D[CB][CB + 1];
  __shared__ float red[GEMM_THREADS];
  __shared__ float col[2][2 * CB];
  const RefreshMat m = rm[blockIdx.x];
  const int r = m.r;
  if (J0 >= r) return;
  float* C = m.C;
  const int tid = threadIdx.x;
  float floor_pivot;
  if (J0 == 0) {
    float tr = 0.f;
    for (int i = tid; i < r; i += GEMM_THREADS) tr += __ldcg(C + (long long)i * r + i);
    red[tid] = tr;
    __syncthreads();
    for (int o = GEMM_THREADS / 2; o > 0; o >>= 1) {
      if (tid < o) red[tid] += red[tid + o];
      __syncthreads();
    }
    const float mean_diag = red[0] / (float)r;
    const float shift = shift_rel * mean_diag;
    floor_pivot = fmaxf(1e-30f, 1e-12f * mean_diag);
    if (tid == 0) m.info[0] = floor_pivot;
    for (int i = tid; i < r; i += GEMM_THREADS) C[(long long)i * r + i] += shift;
    __syncthreads();                       // this block reads its own writes back below
  } else {
    floor_pivot = m.info[0];
  }
  const int jb = min(CB, r - J0);
  // (loads through __ldcg: known to be global, so they can overlap across the stores to shared memory)
#pragma unroll
  for (int e = tid; e < CB * CB; e += GEMM_THREADS) {
    const int i = e / CB, j = e % CB;
    D[i][j] = (i < jb && j < jb) ? __ldcg(C + (long long)(J0 + i) * r + J0 + j) : (i == j ? 1.f : 0.f);
  }
  if (tid < 2 * CB) { col[0][tid] = 0.f; col[1][tid] = 0.f; }
  __syncthreads();
  // Thread i < CB keeps row i in registers, shifted left by one entry per step so that the loop body
  // is the same for every step: at step k, a[j] is the entry of column k + j.  Every row hands its
  // entry of column k to the others through col[] (two buffers in turn; their upper halves stay
  // zero), forms the pivot's root, scales its entry and updates the rest of its row.  Entries right
  // of the diagonal are updated too: they are the mirror images and are never stored.  The two warps
  // that work meet at a barrier of their own.
  if (tid < CB) {
    float a[CB];
#pragma unroll
    for (int j = 0; j < CB; ++j) a[j] = D[tid][j];
#pragma unroll 1
    for (int k = 0; k < CB; ++k) {
      float* ck = col[k & 1];
      ck[tid] = a[0];
      asm volatile("bar.sync 1, %0;" ::"n"(CB) : "memory");
      float pv = ck[k];
      if (!(pv > floor_pivot) || !isfinite(pv)) {
        if (tid == k && k < jb) atomicOr(status, DEV_STATUS_NONFINITE);
        pv = floor_pivot;
      }
      const float s = sqrtf(pv), rs = 1.f / s;
      const float lik = (tid == k) ? s : a[0] * rs;
      D[tid][k] = lik;
#pragma unroll
      for (int j = 1; j < CB; ++j) a[j - 1] = a[j] - lik * (ck[k + j] * rs);
      a[CB - 1] = 0.f;
    }
  }
  __syncthreads();
  for (int e = tid; e < jb * jb; e += GEMM_THREADS) {
    const int i = e / jb, j = e % jb;
    if (j <= i) C[(long long)(J0 + i) * r + J0 + j] = D[i][j];
  }
}

// x <- x L^-T for one row x of CB entries held in registers.  Rows [0, CB) of DT hold the lower
// triangular L (the identity past the matrix's end), rows [CB, 2 CB) zeros.  The row moves left by one
// entry per step and the finished entry comes back in at the right end, so that the loop body is the
// same for every step and the row ends up in order; the zeros are what the entries that are already
// final meet.
__device__ __forceinline__ void solve_row_shifting(float (&a)[CB], const float (*DT)[CB + 1]) {
#pragma unroll 1
  for (int c = 0; c < CB; ++c) {
    const float x = a[0] / DT[c][c];
#pragma unroll
    for (int j = 1; j < CB; ++j) a[j - 1] = a[j] - x * DT[c + j][c];
    a[CB - 1] = x;
  }
}

// Rows below the diagonal block: one block of CB threads per CB rows (tiles_per_matrix of them per
// matrix); a thread is a column while loading and storing, a row while solving x <- x L_JJ^-T
// (solve_row_shifting).
__global__ void __launch_bounds__(CB)
k_chol_panel(const RefreshMat* __restrict__ rm, int J0, int tiles_per_matrix) {
  __shared__ float DT[2 * CB][CB + 1];    // rows < CB: L_JJ (identity past the matrix's end); the rest: the
                                          // tile on its way in and out, zeros during the solve
  const RefreshMat m = rm[blockIdx.x / tiles_per_matrix];
  const int r = m.r;
  const int jb = min(CB, r - J0);
  const int I0 = J0 + CB + (blockIdx.x % tiles_per_matrix) * CB;
  if (J0 >= r || I0 >= r) return;
  float* C = m.C;
  const int tid = threadIdx.x;
#pragma unroll 16
  for (int i = 0; i < CB; ++i) {
    DT[i][tid] = (i < jb && tid < jb) ? __ldcg(C + (long long)(J0 + i) * r + J0 + tid) : (i == tid ? 1.f : 0.f);
    DT[CB + i][tid] = (I0 + i < r && tid < jb) ? __ldcg(C + (long long)(I0 + i) * r + J0 + tid) : 0.f;
  }
  __syncthreads();
  float a[CB];
#pragma unroll
  for (int j = 0; j < CB; ++j) a[j] = DT[CB + tid][j];
  __syncthreads();
#pragma unroll
  for (int i = 0; i < CB; ++i) DT[CB + i][tid] = 0.f;
  __syncthreads();
  solve_row_shifting(a, DT);
  __syncthreads();
#pragma unroll
  for (int j = 0; j < CB; ++j) DT[CB + tid][j] = a[j];
  __syncthreads();
#pragma unroll 16
  for (int i = 0; i < CB; ++i)
    if (I0 + i < r && tid < jb) C[(long long)(I0 + i) * r + J0 + tid] = DT[CB + i][tid];
}

// Trailing update on the 128 x 128 tiles (I >= K) of the part below and right of the panel.
__global__ void __launch_bounds__(GEMM_THREADS, 2)
k_chol_update(const RefreshMat* __restrict__ rm, int J0, int nt) {
  __shared__ __align__(16) float As[TK][SIMT_TILE + 4];
  __shared__ __align__(16) float Bs[TK][SIMT_TILE + 4];
  const int per = nt * (nt + 1) / 2;
  const RefreshMat m = rm[blockIdx.x / per];
  const int r = m.r;
  if (J0 + CB >= r) return;
  int p = blockIdx.x % per, ti = 0;
  while (p > ti) { p -= ti + 1; ++ti; }        // tile row ti, tile column p <= ti
  const int first = ((J0 + CB) / SIMT_TILE) * SIMT_TILE;      // tiles start at a multiple of 128 at or below the panel's end
  const int I0 = first + ti * SIMT_TILE, K0 = first + p * SIMT_TILE;
  if (I0 >= r) return;
  float* C = m.C;
  const int jb = min(CB, r - J0);
  float acc[4 * SIMT_Q][4 * SIMT_Q] = {};
  // A(i, k) = C[i][J0 + k], B(k, j) = C[j][J0 + k]
  gemm_tile<SIMT_Q, float, float>(C + J0, r, 1, C + J0, 1, r, r, r, jb, I0, K0, acc, As, Bs);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int lo = J0 + CB;                      // only rows and columns past the panel change
  if (r % 4 == 0) {
    // Four rows at a time: all their loads first, then the stores (a load after a store to the same
    // array would have to wait for it).  A group of four columns is inside the matrix or outside it
    // as a whole; entries that must not change (above the diagonal, before the panel's end) get
    // their old value back, and no other block touches this tile.
#pragma unroll
    for (int xb = 0; xb < 4 * SIMT_Q; xb += 4) {
      float4 c[4][SIMT_Q];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int i = I0 + tile_coord(ty, xb + x);
#pragma unroll
        for (int q = 0; q < SIMT_Q; ++q) {
          const int j = K0 + tile_coord(tx, 4 * q);
          c[x][q] = (i < r && j < r) ? __ldcg(reinterpret_cast<const float4*>(C + (long long)i * r + j))
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int i = I0 + tile_coord(ty, xb + x);
        if (i >= r || i < lo) continue;
#pragma unroll
        for (int q = 0; q < SIMT_Q; ++q) {
          const int j = K0 + tile_coord(tx, 4 * q);
          if (j >= r || j > i || j + 3 < lo) continue;
          float4 v = c[x][q];
          if (j >= lo && j <= i) v.x -= acc[xb + x][4 * q];
          if (j + 1 >= lo && j + 1 <= i) v.y -= acc[xb + x][4 * q + 1];
          if (j + 2 >= lo && j + 2 <= i) v.z -= acc[xb + x][4 * q + 2];
          if (j + 3 >= lo && j + 3 <= i) v.w -= acc[xb + x][4 * q + 3];
          *reinterpret_cast<float4*>(C + (long long)i * r + j) = v;
        }
      }
    }
    return;
  }
#pragma unroll
  for (int x = 0; x < 4 * SIMT_Q; ++x) {
    const int i = I0 + tile_coord(ty, x);
    if (i >= r || i < lo) continue;
#pragma unroll
    for (int y = 0; y < 4 * SIMT_Q; ++y) {
      const int j = K0 + tile_coord(tx, y);
      if (j <= i && j >= lo) C[(long long)i * r + j] -= acc[x][y];
    }
  }
}

// ------------------------------------------------------------------ X <- X L^-T
// One block per tile of 64 rows of X (rows x r, in place).  For each 64-wide
// block column J: X_J = (X_J - X_{<J} L[J, <J]^T) L_JJ^-T.
// tri: X starts as the identity (the solve that produces L^-T itself).  The result is upper
// triangular and stays so on the way, so a row tile starts at its own diagonal block and its
// products run over the columns from there on: a third of the work.
struct TrsmDesc { float* X; const float* L; int rows, r; int tri; };

__global__ void __launch_bounds__(GEMM_THREADS)
k_trsm_rows(const TrsmDesc* __restrict__ descs, int ndesc, const int* __restrict__ tile_start) {
  static_assert(TM == CB, "one row of the tile per solving thread");
  __shared__ __align__(16) float As[TK][TM + 4];
  __shared__ __align__(16) float Bs[TK][TN + 4];
  __shared__ float DT[2 * CB][CB + 1];         // rows < CB: L_JJ; the rest: the tile on its way in and out,
                                               // zeros during the solve (solve_row_shifting)
  const int p = find_matrix(tile_start, ndesc, blockIdx.x);
  const TrsmDesc t = descs[p];
  const int I0 = (blockIdx.x - tile_start[p]) * TM;
  const int r = t.r;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int K0 = t.tri ? I0 : 0;               // first column of X that can be non-zero in these rows
  for (int J0 = K0; J0 < r; J0 += CB) {
    const int jb = min(CB, r - J0);
    float acc[4][4] = {};
    gemm_tile<1, float, float>(t.X + K0, r, 1, t.L + K0, 1, r, t.rows, J0 + jb, J0 - K0, I0, J0, acc, As, Bs);
    float xin[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        const int il = ty * 4 + x, jl = tx * 4 + y;
        xin[x][y] = (I0 + il < t.rows && jl < jb) ? __ldcg(t.X + (long long)(I0 + il) * r + J0 + jl) : 0.f;
      }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        const int il = ty * 4 + x, jl = tx * 4 + y;
        DT[CB + il][jl] = (I0 + il < t.rows && jl < jb) ? xin[x][y] - acc[x][y] : 0.f;
      }
#pragma unroll
    for (int e = tid; e < CB * CB; e += GEMM_THREADS) {
      const int i = e / CB, j = e % CB;
      DT[i][j] = (i < jb && j < jb) ? __ldcg(t.L + (long long)(J0 + i) * r + J0 + j) : (i == j ? 1.f : 0.f);
    }
    __syncthreads();
    float a[CB];
    if (tid < TM) {
#pragma unroll
      for (int j = 0; j < CB; ++j) a[j] = DT[CB + tid][j];
    }
    __syncthreads();
    for (int e = tid; e < CB * CB; e += GEMM_THREADS) DT[CB + e / CB][e % CB] = 0.f;
    __syncthreads();
    if (tid < TM) solve_row_shifting(a, DT);
    __syncthreads();
    if (tid < TM) {
#pragma unroll
      for (int j = 0; j < CB; ++j) DT[CB + tid][j] = a[j];
    }
    __syncthreads();
    for (int e = tid; e < TM * CB; e += GEMM_THREADS) {
      const int i = e / CB, j = e % CB;
      if (I0 + i < t.rows && j < jb) t.X[(long long)(I0 + i) * r + J0 + j] = DT[CB + i][j];
    }
    __syncthreads();                           // the next block column's product reads these columns
  }
}

__global__ void __launch_bounds__(256)
k_store_projection(const RefreshMat* __restrict__ rm) {
  const RefreshMat m = rm[blockIdx.y];
  const long long total = (long long)m.d * m.r;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    if (m.bf16) ((__nv_bfloat16*)m.P)[i] = __float2bfloat16_rn(m.Y[i]);
    else ((float*)m.P)[i] = m.Y[i];
    if (m.out32) m.out32[i] = m.Y[i];
  }
}

// bf16 operands of the next tensor-core product: hi = bf16(x) and, if asked for, lo = bf16(x - hi)
// (which = 0: Y, 1: Z, 2: U).
__global__ void __launch_bounds__(256)
k_split_bf16(const RefreshMat* __restrict__ rm, int which, int with_lo) {
  const RefreshMat m = rm[blockIdx.y];
  if (!m.tc) return;
  const float* src = which == 0 ? m.Y : which == 1 ? m.Z : m.U;
  __nv_bfloat16* hi = which == 0 ? m.Yb : which == 1 ? m.Zb : m.Ub;
  __nv_bfloat16* lo = which == 0 ? m.Yl : which == 1 ? m.Zl : m.Ul;
  const long long rows = which == 0 ? m.d : which == 1 ? m.l : m.r;
  const long long quads = rows * m.r / 4;      // r is a multiple of 128
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < quads;
       q += (long long)gridDim.x * blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(src)[q];
    const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<const unsigned*>(&a); u.y = *reinterpret_cast<const unsigned*>(&b);
    reinterpret_cast<uint2*>(hi)[q] = u;
    if (with_lo) {
      const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
      const __nv_bfloat162 c = __floats2bfloat162_rn(v.x - fa.x, v.y - fa.y), e = __floats2bfloat162_rn(v.z - fb.x, v.w - fb.y);
      uint2 w;
      w.x = *reinterpret_cast<const unsigned*>(&c); w.y = *reinterpret_cast<const unsigned*>(&e);
      reinterpret_cast<uint2*>(lo)[q] = w;
    }
  }
}

// U <- identity (r x r); the triangular-solve kernel then turns it into L^-T.
__global__ void __launch_bounds__(256)
k_identity(const RefreshMat* __restrict__ rm) {
  const RefreshMat m = rm[blockIdx.y];
  if (!m.tc) return;
  const long long total = (long long)m.r * m.r;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x)
    m.U[i] = (i / m.r == i % m.r) ? 1.f : 0.f;
}

// descriptor tables of a chunk: per-matrix entries plus alignment slack
constexpr size_t TABLE_PER_MATRIX = 1024;
constexpr size_t TABLE_SLACK = 16 * 1024;
static_assert(sizeof(RefreshMat) + 4 * sizeof(GemmDesc) + 3 * sizeof(TrsmDesc) + 10 * sizeof(int) <= TABLE_PER_MATRIX, "table allowance");

}  // namespace

// bf16 matrices that TMA can read in place: their products run on the tensor cores
static bool refresh_on_tc(const fira_matrix_desc& d) {
  return d.dtype == FIRA_BF16 && tc_supported(d) && tc_rows_aligned(d);   // the refresh only reads G
}

// The kinds of tensor-core jobs of one matrix: A Z and A^T Y (plain and with a split iterate), the
// two Gram products and the two applications of L^-T, each with split operands (three k-segments,
// for the basis that is kept) and with plain bf16 operands (one segment, for the intermediate
// iterates, which the next product rounds to bf16 anyway and which only have to stay well
// conditioned).
enum { JOB_AZ = 0, JOB_AZ_SPLIT, JOB_ATY, JOB_ATY_SPLIT, JOB_GRAM_Y, JOB_GRAM_Z, JOB_APPLY_Y, JOB_APPLY_Z,
       JOB_GRAM_Y1, JOB_GRAM_Z1, JOB_APPLY_Y1, JOB_APPLY_Z1, JOB_KINDS };

static TcGemmJob refresh_job(const fira_matrix_desc& dsc, int kind) {
  TcGemmJob j;
  memset(&j, 0, sizeof(j));
  const int d = std::min(dsc.m, dsc.n), l = std::max(dsc.m, dsc.n);
  const bool left = dsc.m <= dsc.n;
  j.r = dsc.r;
  switch (kind) {
    case JOB_AZ: case JOB_AZ_SPLIT: case JOB_ATY: case JOB_ATY_SPLIT: {
      const bool az = kind == JOB_AZ || kind == JOB_AZ_SPLIT;
      j.m = dsc.m; j.n = dsc.n; j.ld = dsc.ld ? dsc.ld : dsc.n;
      j.mn_major = az ? !left : left;      // A Z: rows d, k = l;  A^T Y: rows l, k = d
      if (kind == JOB_AZ_SPLIT || kind == JOB_ATY_SPLIT) { j.nseg = 2; j.asel = 0u; j.bsel = 2u; }   // A hi, A lo(iterate)
      break;
    }
    case JOB_GRAM_Y: case JOB_GRAM_Z: case JOB_GRAM_Y1: case JOB_GRAM_Z1:   // C[i][j] = sum_k X[k][i] X[k][j]: "G" = X as [k][i]
      j.m = (kind == JOB_GRAM_Y || kind == JOB_GRAM_Y1) ? d : l; j.n = dsc.r; j.ld = dsc.r; j.mn_major = 1;
      if (kind == JOB_GRAM_Y || kind == JOB_GRAM_Z) { j.nseg = 3; j.asel = 4u; j.bsel = 2u; }   // hi hi, hi lo, lo hi
      break;
    default:                               // X[i][j] = sum_k X[i][k] U[k][j]: "G" = X as [i][k]
      j.m = (kind == JOB_APPLY_Y || kind == JOB_APPLY_Y1) ? d : l; j.n = dsc.r; j.ld = dsc.r; j.mn_major = 0;
      if (kind == JOB_APPLY_Y || kind == JOB_APPLY_Z) { j.nseg = 3; j.asel = 4u; j.bsel = 2u; }
      break;
  }
  return j;
}

static size_t refresh_data_bytes(const fira_matrix_desc& d) {
  const size_t dd = std::min(d.m, d.n), ll = std::max(d.m, d.n), r = d.r;
  size_t b = align_up(dd * r * 4) + align_up(ll * r * 4) + align_up(r * r * 4) + 256;
  if (refresh_on_tc(d)) {
    b += align_up(r * r * 4) + 2 * (align_up(dd * r * 2) + align_up(ll * r * 2) + align_up(r * r * 2));
    for (int k = 0; k < JOB_KINDS; ++k) { const TcGemmJob j = refresh_job(d, k); b += tc_gemm_table_bytes(&j, 1); }
  }
  return b;
}

size_t refresh_bytes_per_matrix(const fira_matrix_desc& d) {
  return refresh_data_bytes(d) + TABLE_PER_MATRIX + TABLE_SLACK;
}

#define RF_CUDA(call)                                                          \
  do {                                                                         \
    cudaError_t e_ = (call);                                                   \
    if (e_ != cudaSuccess) {                                                   \
      set_error(std::string(#call) + ": " + cudaGetErrorString(e_));           \
      return FIRA_ERR_CUDA;                                                    \
    }                                                                          \
  } while (0)

// Refreshes the matrices of `which` in chunks that fit the work area.  The work
// area is shared with the step's scratch, whose contents are dead between steps.
// basis_out (may be null): per matrix index an optional device pointer that receives the kept
// basis in fp32 (d x r) before it is rounded to the storage type.
fira_status refresh_impl(fira_ctx* c, const void* const* G_dev, const std::vector<int>& which,
                         uint64_t seed, int iters, float* const* basis_out, const RefreshTarget* target) {
  if (iters < 0) iters = 4;
  RefreshTarget own;
  own.work_base = c->work_base; own.work_bytes = c->work_bytes; own.stream = c->stream;
  const RefreshTarget& tg = target ? *target : own;
  if (!tg.P_out) c->proj_weights_dirty = true;
  cudaStream_t st = tg.stream;
  size_t pos = 0;
  while (pos < which.size()) {
    // ---- carve a chunk: as many matrices as fit (data regions first, then tables)
    std::vector<size_t> offs;
    size_t off = 0, q = pos;
    for (; q < which.size(); ++q) {
      const size_t data = refresh_data_bytes(c->descs[which[q]]);
      if (off + data + (q - pos + 1) * TABLE_PER_MATRIX + TABLE_SLACK > tg.work_bytes) break;
      offs.push_back(off);
      off += data;
    }
    if (q == pos) { set_error("scratch buffer too small for the projection refresh"); return FIRA_ERR_WORKSPACE_TOO_SMALL; }
    const int nm = (int)(q - pos);
    std::vector<RefreshMat> rms;
    size_t data_end = 0;
    for (int a = 0; a < nm; ++a) {
      const int idx = which[pos + a];
      const MatDev& mt = c->mats[idx];
      RefreshMat rm;
      memset(&rm, 0, sizeof(rm));
      rm.G = G_dev[idx]; rm.P = tg.P_out ? tg.P_out[idx] : mt.P;
      rm.out32 = basis_out ? basis_out[idx] : nullptr;
      char* base = tg.work_base + offs[a];
      const size_t r = mt.r;
      rm.Y = (float*)base; base += align_up((size_t)mt.d * r * 4);
      rm.Z = (float*)base; base += align_up((size_t)mt.l * r * 4);
      rm.C = (float*)base; base += align_up(r * r * 4);
      rm.info = (float*)base; base += 256;
      rm.tc = refresh_on_tc(c->descs[idx]) ? 1 : 0;
      if (rm.tc) {
        rm.U = (float*)base; base += align_up(r * r * 4);
        rm.Yb = (__nv_bfloat16*)base; base += align_up((size_t)mt.d * r * 2);
        rm.Yl = (__nv_bfloat16*)base; base += align_up((size_t)mt.d * r * 2);
        rm.Zb = (__nv_bfloat16*)base; base += align_up((size_t)mt.l * r * 2);
        rm.Zl = (__nv_bfloat16*)base; base += align_up((size_t)mt.l * r * 2);
        rm.Ub = (__nv_bfloat16*)base; base += align_up(r * r * 2);
        rm.Ul = (__nv_bfloat16*)base; base += align_up(r * r * 2);
      }
      data_end = std::max(data_end, (size_t)(base - tg.work_base));
      rm.ld = mt.ld; rm.d = mt.d; rm.l = mt.l; rm.r = mt.r; rm.left = mt.left; rm.bf16 = mt.bf16;
      rm.key = seed * 0x9E3779B97F4A7C15ull + (unsigned long long)idx * 0xD1B54A32D192ED03ull + 1ull;
      rms.push_back(rm);
    }
    // ---- descriptor tables of the CUDA-core kernels: AZ->Y, A^T Y->Z, Y^T Y->C, Z^T Z->C, trsm(Y), trsm(Z)
    // for the matrices that stay there; trsm(U) for the others
    std::vector<GemmDesc> gAZ, gAtY, gYY, gZZ;
    std::vector<TrsmDesc> tY, tZ, tU;
    std::vector<int> sAZ{0}, sAtY{0}, sYY{0}, sTY{0}, sTZ{0}, sTU{0};
    auto tiles = [](int I, int J) { return simt_tiles(I) * simt_tiles(J); };
    std::vector<TcGemmJob> jobs[JOB_KINDS];
    for (size_t a = 0; a < rms.size(); ++a) {
      const RefreshMat& m = rms[a];
      if (m.tc) {
        const fira_matrix_desc& dd = c->descs[which[pos + a]];
        for (int k = 0; k < JOB_KINDS; ++k) {
          TcGemmJob j = refresh_job(dd, k);
          switch (k) {
            case JOB_AZ: case JOB_AZ_SPLIT: j.G = m.G; j.B = m.Zb; j.B_lo = k == JOB_AZ_SPLIT ? m.Zl : nullptr; j.C = m.Y; break;
            case JOB_ATY: case JOB_ATY_SPLIT: j.G = m.G; j.B = m.Yb; j.B_lo = k == JOB_ATY_SPLIT ? m.Yl : nullptr; j.C = m.Z; break;
            case JOB_GRAM_Y: j.G = m.Yb; j.G_lo = m.Yl; j.B = m.Yb; j.B_lo = m.Yl; j.C = m.C; break;
            case JOB_GRAM_Z: j.G = m.Zb; j.G_lo = m.Zl; j.B = m.Zb; j.B_lo = m.Zl; j.C = m.C; break;
            case JOB_APPLY_Y: j.G = m.Yb; j.G_lo = m.Yl; j.B = m.Ub; j.B_lo = m.Ul; j.C = m.Y; break;
            case JOB_APPLY_Z: j.G = m.Zb; j.G_lo = m.Zl; j.B = m.Ub; j.B_lo = m.Ul; j.C = m.Z; break;
            case JOB_GRAM_Y1: j.G = m.Yb; j.B = m.Yb; j.C = m.C; break;
            case JOB_GRAM_Z1: j.G = m.Zb; j.B = m.Zb; j.C = m.C; break;
            case JOB_APPLY_Y1: j.G = m.Yb; j.B = m.Ub; j.C = m.Y; break;
            default: j.G = m.Zb; j.B = m.Ub; j.C = m.Z; break;
          }
          jobs[k].push_back(j);
        }
        tU.push_back(TrsmDesc{m.U, m.C, m.r, m.r, 1}); sTU.push_back(sTU.back() + (m.r + TM - 1) / TM);
        continue;
      }
      GemmDesc g;
      // Y[d][j] = sum_l A(d,l) Z[l][j]
      g.A = m.G; g.a_bf16 = m.bf16;
      g.sAi = m.left ? m.ld : 1; g.sAk = m.left ? 1 : m.ld;
      g.B = m.Z; g.sBk = m.r; g.sBj = 1; g.C = m.Y; g.sCi = m.r; g.I = m.d; g.J = m.r; g.K = m.l;
      gAZ.push_back(g); sAZ.push_back(sAZ.back() + tiles(g.I, g.J));
      // Z[l][j] = sum_d A(d,l) Y[d][j]
      g.sAi = m.left ? 1 : m.ld; g.sAk = m.left ? m.ld : 1;
      g.B = m.Y; g.C = m.Z; g.I = m.l; g.K = m.d;
      gAtY.push_back(g); sAtY.push_back(sAtY.back() + tiles(g.I, g.J));
      // C = Y^T Y and C = Z^T Z
      g.a_bf16 = 0; g.sAi = 1; g.sAk = m.r; g.sBk = m.r; g.sBj = 1; g.C = m.C; g.sCi = m.r; g.I = m.r; g.J = m.r;
      g.A = m.Y; g.B = m.Y; g.K = m.d; gYY.push_back(g);
      g.A = m.Z; g.B = m.Z; g.K = m.l; gZZ.push_back(g);
      sYY.push_back(sYY.back() + tiles(m.r, m.r));
      tY.push_back(TrsmDesc{m.Y, m.C, m.d, m.r, 0}); sTY.push_back(sTY.back() + (m.d + TM - 1) / TM);
      tZ.push_back(TrsmDesc{m.Z, m.C, m.l, m.r, 0}); sTZ.push_back(sTZ.back() + (m.l + TM - 1) / TM);
    }
    char* tp = tg.work_base + align_up(data_end);
    cudaError_t cerr = cudaSuccess;
    auto put = [&](const void* src, size_t bytes) -> char* {
      char* dst = tp;
      if (bytes == 0) return dst;
      if ((size_t)(tp + align_up(bytes) - tg.work_base) > tg.work_bytes) { cerr = cudaErrorInvalidValue; return dst; }
      cudaError_t e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st);
      if (e != cudaSuccess) cerr = e;
      tp += align_up(bytes);
      return dst;
    };
    const RefreshMat* rm_dev = (const RefreshMat*)put(rms.data(), rms.size() * sizeof(RefreshMat));
    const GemmDesc* dAZ = (const GemmDesc*)put(gAZ.data(), gAZ.size() * sizeof(GemmDesc));
    const GemmDesc* dAtY = (const GemmDesc*)put(gAtY.data(), gAtY.size() * sizeof(GemmDesc));
    const GemmDesc* dYY = (const GemmDesc*)put(gYY.data(), gYY.size() * sizeof(GemmDesc));
    const GemmDesc* dZZ = (const GemmDesc*)put(gZZ.data(), gZZ.size() * sizeof(GemmDesc));
    const TrsmDesc* dTY = (const TrsmDesc*)put(tY.data(), tY.size() * sizeof(TrsmDesc));
    const TrsmDesc* dTZ = (const TrsmDesc*)put(tZ.data(), tZ.size() * sizeof(TrsmDesc));
    const TrsmDesc* dTU = (const TrsmDesc*)put(tU.data(), tU.size() * sizeof(TrsmDesc));
    const int* dsAZ = (const int*)put(sAZ.data(), sAZ.size() * sizeof(int));
    const int* dsAtY = (const int*)put(sAtY.data(), sAtY.size() * sizeof(int));
    const int* dsYY = (const int*)put(sYY.data(), sYY.size() * sizeof(int));
    const int* dsTY = (const int*)put(sTY.data(), sTY.size() * sizeof(int));
    const int* dsTZ = (const int*)put(sTZ.data(), sTZ.size() * sizeof(int));
    const int* dsTU = (const int*)put(sTU.data(), sTU.size() * sizeof(int));
    if (cerr != cudaSuccess) { set_error(std::string("refresh tables: ") + cudaGetErrorString(cerr)); return FIRA_ERR_CUDA; }
    // tables of the tensor-core jobs (tensor maps and tile records), after the others
    const int ntc = (int)jobs[0].size(), nsimt = nm - ntc;
    char* tab[JOB_KINDS] = {};
    int jtiles[JOB_KINDS] = {};
    if (ntc) {
      for (int k = 0; k < JOB_KINDS; ++k) {
        const size_t bytes = tc_gemm_table_bytes(jobs[k].data(), ntc);
        if ((size_t)(tp + bytes - tg.work_base) > tg.work_bytes) {
          set_error("scratch buffer too small for the projection refresh"); return FIRA_ERR_WORKSPACE_TOO_SMALL;
        }
        tab[k] = tp;
        const fira_status ps = tc_gemm_prepare(c, jobs[k].data(), ntc, tab[k], bytes, &jtiles[k], st);
        if (ps != FIRA_OK) return ps;
        tp += bytes;
      }
    }
    int rmax = 0;
    for (const RefreshMat& m : rms) rmax = std::max(rmax, m.r);
    const dim3 ew_grid(296, nm);      // element-wise helpers: every matrix of the chunk, tc ones act
    // A Z -> Y and A^T Y -> Z.  precise: the iterate enters with its bf16 remainder as a second k-segment.
    auto product = [&](bool az, bool precise) -> fira_status {
      if (nsimt) {
        if (az) k_rgemm<<<sAZ.back(), GEMM_THREADS, 0, st>>>(dAZ, nsimt, dsAZ);
        else k_rgemm<<<sAtY.back(), GEMM_THREADS, 0, st>>>(dAtY, nsimt, dsAtY);
      }
      if (ntc) {
        k_split_bf16<<<ew_grid, 256, 0, st>>>(rm_dev, az ? 1 : 0, precise ? 1 : 0);
        const int k = az ? (precise ? JOB_AZ_SPLIT : JOB_AZ) : (precise ? JOB_ATY_SPLIT : JOB_ATY);
        return tc_gemm_run(c, tab[k], ntc, jtiles[k], st);
      }
      return FIRA_OK;
    };
    // CholeskyQR of Y (y = true) or Z; the second pass brings the basis to fp32 orthonormality and is
    // needed only for the basis that is kept: one pass (deviation about cond^2 times the product's
    // precision) keeps an intermediate iterate well conditioned, which is all the next product asks.
    // precise: split operands (the basis that is kept); otherwise plain bf16 operands.
    auto orth = [&](bool y, int passes, bool precise) -> fira_status {
      const int kg = y ? (precise ? JOB_GRAM_Y : JOB_GRAM_Y1) : (precise ? JOB_GRAM_Z : JOB_GRAM_Z1);
      const int ka = y ? (precise ? JOB_APPLY_Y : JOB_APPLY_Y1) : (precise ? JOB_APPLY_Z : JOB_APPLY_Z1);
      for (int pass = 0; pass < passes; ++pass) {
        if (nsimt) k_rgemm<<<sYY.back(), GEMM_THREADS, 0, st>>>(y ? dYY : dZZ, nsimt, dsYY);
        if (ntc) {
          k_split_bf16<<<ew_grid, 256, 0, st>>>(rm_dev, y ? 0 : 1, precise ? 1 : 0);
          const fira_status gs = tc_gemm_run(c, tab[kg], ntc, jtiles[kg], st);
          if (gs != FIRA_OK) return gs;
        }
        for (int J0 = 0; J0 < rmax; J0 += CB) {
          k_chol_diag<<<nm, GEMM_THREADS, 0, st>>>(rm_dev, J0, pass == 0 ? 1e-6f : 0.f, c->status_dev);
          if (J0 + CB < rmax) {
            k_chol_panel<<<nm * ((rmax - J0 - CB + 63) / 64), 64, 0, st>>>(rm_dev, J0, (rmax - J0 - CB + 63) / 64);
            const int nt = (rmax - ((J0 + CB) / SIMT_TILE) * SIMT_TILE + SIMT_TILE - 1) / SIMT_TILE;
            k_chol_update<<<nm * (nt * (nt + 1) / 2), GEMM_THREADS, 0, st>>>(rm_dev, J0, nt);
          }
        }
        if (nsimt) {
          if (y) k_trsm_rows<<<sTY.back(), GEMM_THREADS, 0, st>>>(dTY, nsimt, dsTY);
          else k_trsm_rows<<<sTZ.back(), GEMM_THREADS, 0, st>>>(dTZ, nsimt, dsTZ);
        }
        if (ntc) {
          k_identity<<<ew_grid, 256, 0, st>>>(rm_dev);
          k_trsm_rows<<<sTU.back(), GEMM_THREADS, 0, st>>>(dTU, ntc, dsTU);      // U = L^-T
          k_split_bf16<<<ew_grid, 256, 0, st>>>(rm_dev, 2, precise ? 1 : 0);
          const fira_status as = tc_gemm_run(c, tab[ka], ntc, jtiles[ka], st);
          if (as != FIRA_OK) return as;
        }
      }
      return FIRA_OK;
    };
    k_gauss<<<ew_grid, 256, 0, st>>>(rm_dev);
    fira_status prs = product(true, iters == 0);
    if (prs == FIRA_OK) prs = orth(true, iters == 0 ? 2 : 1, iters == 0);
    for (int it = 0; it < iters && prs == FIRA_OK; ++it) {
      const bool last = it + 1 == iters;
      prs = product(false, last);
      if (prs == FIRA_OK) prs = orth(false, 1, last);
      if (prs == FIRA_OK) prs = product(true, last);
      if (prs == FIRA_OK) prs = orth(true, last ? 2 : 1, last);
    }
    if (prs != FIRA_OK) return prs;
    k_store_projection<<<ew_grid, 256, 0, st>>>(rm_dev);
    RF_CUDA(cudaGetLastError());
    // the next chunk reuses the work area, and the host tables above die here
    RF_CUDA(cudaStreamSynchronize(st));
    pos = q;
  }
  return FIRA_OK;
}

}  // namespace fira
