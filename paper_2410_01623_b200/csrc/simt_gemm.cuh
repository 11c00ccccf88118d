// Shared-memory tiled fp32 product on the CUDA cores, with arbitrary element strides for both
// operands: a block of 256 threads computes a (64 Q) x (64 Q) tile in slabs of 16 along k.
// Used by the fp32 step kernels and by the projection refresh.  The next slab is fetched into
// registers while the current one is multiplied; where an operand is contiguous along one of the
// slab's directions and suitably aligned, four elements move per load.  The operands are read with
// plain loads (no read-only cache path), so a kernel may read back what it wrote earlier after a
// barrier.
#pragma once
#include "common.cuh"

namespace fira {

constexpr int TM = 64, TN = 64, TK = 16;    // the Q = 1 tile
constexpr int GEMM_THREADS = 256;
constexpr int SIMT_Q = 2;                   // tile factor of the step and refresh products (128 x 128)
constexpr int SIMT_TILE = 64 * SIMT_Q;
inline int simt_tiles(long long extent) { return (int)((extent + SIMT_TILE - 1) / SIMT_TILE); }

// Row (or column) of accumulator index x within a tile: quadrant x / 4, then the thread's 4.
__device__ __forceinline__ int tile_coord(int t16, int x) { return (x >> 2) * 64 + t16 * 4 + (x & 3); }

namespace detail {

__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
  const float4 u = *reinterpret_cast<const float4*>(p);
  v[0] = u.x; v[1] = u.y; v[2] = u.z; v[3] = u.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(u.x << 16); v[1] = __uint_as_float(u.x & 0xffff0000u);
  v[2] = __uint_as_float(u.y << 16); v[3] = __uint_as_float(u.y & 0xffff0000u);
}

// One operand slab S[k][x] = Op(x0 + x, k0 + k), Op(x, k) = base[x * sx + k * sk], zero outside
// X x K.  Each thread owns Q groups of four elements that are consecutive along x (when sx == 1)
// or along k (otherwise).
template <int Q, typename T>
struct Slab {
  float v[Q][4];
  const T* base;
  long long sx, sk;
  int X, K, x0;
  bool along_x, vec;

  __device__ __forceinline__ void init(const T* b, long long sx_, long long sk_, int X_, int K_, int x0_) {
    base = b; sx = sx_; sk = sk_; X = X_; K = K_; x0 = x0_;
    along_x = (sx == 1);
    const long long other = along_x ? sk : sx;
    // a group is one aligned 4-element vector when the base is aligned and the other stride keeps it so
    vec = (along_x || sk == 1) && (other % 4 == 0) &&
          (reinterpret_cast<unsigned long long>(b) % (4 * sizeof(T)) == 0) && (!along_x || x0 % 4 == 0);
  }
  __device__ __forceinline__ void coords(int q, int& x, int& k) const {
    const int e = (threadIdx.x + GEMM_THREADS * q) * 4;
    if (along_x) { x = e % (64 * Q); k = e / (64 * Q); } else { k = e % TK; x = e / TK; }
  }
  __device__ __forceinline__ void load(int k0) {
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      int x, k;
      coords(q, x, k);
      const int gx = x0 + x, gk = k0 + k;
      const T* p = base + (long long)gx * sx + (long long)gk * sk;
      const bool all_in = along_x ? (gx + 3 < X && gk < K) : (gx < X && gk + 3 < K);
      if (vec && all_in) {
        load4(p, v[q]);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int cx = along_x ? gx + c : gx, ck = along_x ? gk : gk + c;
          v[q][c] = (cx < X && ck < K) ? to_float<T>(p[along_x ? (long long)c : (long long)c * sk]) : 0.f;
        }
      }
    }
  }
  __device__ __forceinline__ void store(float (*S)[64 * Q + 4]) const {
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      int x, k;
      coords(q, x, k);
      if (along_x) {
        *reinterpret_cast<float4*>(&S[k][x]) = make_float4(v[q][0], v[q][1], v[q][2], v[q][3]);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) S[k + c][x] = v[q][c];
      }
    }
  }
};

}  // namespace detail

// acc[x][y] += sum_k A(i0 + tile_coord(ty, x), k) B(k, j0 + tile_coord(tx, y)) over a (64 Q)^2 tile,
// tx = tid % 16, ty = tid / 16.  A(i,k) = A[i*sAi + k*sAk], B(k,j) = B[k*sBk + j*sBj];
// reads outside I x K / K x J give 0.  Ends with a block barrier.
template <int Q, typename TA, typename TB>
__device__ __forceinline__ void gemm_tile(const TA* A, long long sAi, long long sAk,
                                          const TB* B, long long sBk, long long sBj,
                                          int I, int J, int K, int i0, int j0, float (&acc)[4 * Q][4 * Q],
                                          float (*As)[64 * Q + 4], float (*Bs)[64 * Q + 4]) {
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  detail::Slab<Q, TA> sa;
  detail::Slab<Q, TB> sb;
  sa.init(A, sAi, sAk, I, K, i0);
  sb.init(B, sBj, sBk, J, K, j0);
  sa.load(0);
  sb.load(0);
  sa.store(As);
  sb.store(Bs);
  __syncthreads();
  for (int k0 = 0; k0 < K; k0 += TK) {
    const bool more = k0 + TK < K;
    if (more) { sa.load(k0 + TK); sb.load(k0 + TK); }
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float av[4 * Q], bv[4 * Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        const float4 a = *reinterpret_cast<const float4*>(&As[kk][q * 64 + ty * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][q * 64 + tx * 4]);
        av[4 * q] = a.x; av[4 * q + 1] = a.y; av[4 * q + 2] = a.z; av[4 * q + 3] = a.w;
        bv[4 * q] = b.x; bv[4 * q + 1] = b.y; bv[4 * q + 2] = b.z; bv[4 * q + 3] = b.w;
      }
#pragma unroll
      for (int x = 0; x < 4 * Q; ++x)
#pragma unroll
        for (int y = 0; y < 4 * Q; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
    }
    __syncthreads();
    if (more) {
      sa.store(As);
      sb.store(Bs);
      __syncthreads();
    }
  }
}

}  // namespace fira
