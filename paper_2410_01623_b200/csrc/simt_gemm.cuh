// 64 x 64 x 16 shared-memory tiled fp32 product on the CUDA cores, with arbitrary
// element strides for both operands.  Used by the fp32 step kernels and by the
// projection refresh.  The operands are read with plain loads (no read-only
// cache path), so a kernel may read back what it wrote earlier after a barrier.
#pragma once
#include "common.cuh"

namespace fira {

constexpr int TM = 64, TN = 64, TK = 16;
constexpr int GEMM_THREADS = 256;

// acc[x][y] += sum_k A(i0 + ty*4 + x, k) B(k, j0 + tx*4 + y) over a 64 x 64 tile,
// tx = tid % 16, ty = tid / 16.  A(i,k) = A[i*sAi + k*sAk], B(k,j) = B[k*sBk + j*sBj];
// reads outside I x K / K x J give 0.  Ends with a block barrier.
template <typename TA, typename TB>
__device__ __forceinline__ void gemm_tile(const TA* A, long long sAi, long long sAk,
                                          const TB* B, long long sBk, long long sBj,
                                          int I, int J, int K, int i0, int j0, float (&acc)[4][4],
                                          float (*As)[TM + 4], float (*Bs)[TN + 4]) {
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const bool a_i_contig = (sAi == 1);
  const bool b_j_contig = (sBj == 1);
  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int e = tid + GEMM_THREADS * q;
      int i, k;
      if (a_i_contig) { i = e & 63; k = e >> 6; } else { k = e & 15; i = e >> 4; }
      float v = 0.f;
      if (i0 + i < I && k0 + k < K)
        v = to_float<TA>(A[(long long)(i0 + i) * sAi + (long long)(k0 + k) * sAk]);
      As[k][i] = v;
      int j, kb;
      if (b_j_contig) { j = e & 63; kb = e >> 6; } else { kb = e & 15; j = e >> 4; }
      float u = 0.f;
      if (j0 + j < J && k0 + kb < K)
        u = to_float<TB>(B[(long long)(k0 + kb) * sBk + (long long)(j0 + j) * sBj]);
      Bs[kb][j] = u;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w};
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(av[x], bv[y], acc[x][y]);
    }
    __syncthreads();
  }
}

}  // namespace fira
