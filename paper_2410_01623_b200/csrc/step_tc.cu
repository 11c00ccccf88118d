// bf16 tensor-core kernels of the Fira step (Algorithm 1's loop body) for sm_100a:
// TMA-fed tcgen05.mma with fp32 accumulators in tensor memory and fused epilogues,
// grouped over a list of matrices (persistent CTAs walk a static tile list).
//
// l = unprojected index (columns of G when m <= n, rows otherwise), d = projected
// index, Pi = the d x r projection.  Launches per step:
//   k_tc_prep          bias factor sqrt(1-b2^s)/(1-b1^s) per matrix
//   k_tc_project       Rt = G^T Pi on the tensor cores; epilogue: M, V update (Eq. 2-3),
//                      N (Eq. 4), bf16 copies of N and R, per-l partial ||N_l||^2, ||R_l||^2;
//                      ||G_l||^2 from the A stages in shared memory             (for ||S||)
//   k_tc_colfactors    k_l (Eq. 11) and partial sums of ||S||^2 = sum_l k_l^2 (||G_l||^2 - ||R_l||^2)
//   k_finalize         lambda, ||S_prev||, t (Eq. 12)
//   k_tc_form_x        X = a_low N - a_res lambda k_l R  (bf16).  In the plain step the projection
//                      epilogue has written X for lambda = 1 already (see tc_project.cuh) and this
//                      kernel only touches the matrices whose limiter acted (k_tc_fix_x):
//                      X <- lambda X + (1 - lambda) a_low N, N rebuilt from the stored moments
//   k_tc_back_project  D = Pi X on the tensor cores; epilogue: W -= lr (D + a_res lambda k_l G)
//
// ||S_l||^2 = ||G_l - Pi R_l||^2 = ||G_l||^2 - 2 ||R_l||^2 + R_l^T (Pi^T Pi) R_l.  For orthonormal
// columns this is ||G_l||^2 - ||R_l||^2; the stored projection is rounded to bf16, and where its
// columns are concentrated on a few coordinates (outlier columns of G) their norms are off by up
// to 2^-8, which matters because ||S||^2 is a small difference when the subspace holds most of
// the energy.  The kernels therefore use the diagonal of Pi^T Pi: ||S_l||^2 = ||G_l||^2 -
// sum_j (2 - ||pi_j||^2) R_lj^2, with the column norms of the stored projection recomputed
// whenever it changes (k_tc_proj_weights); what is left is the off-diagonal part, which
// averages out.  It only enters the limiter factor lambda and the remembered norm.
//
// Both tensor-core kernels run on CTA pairs (clusters of two, tcgen05 cta_group::2):
// tiles of 256 x BN <= 256 accumulator elements per pair, 64 (one 128-byte swizzle row of
// bf16) deep per pipeline stage; two accumulators of 256 tensor-memory columns alternate so
// that the epilogue of one tile overlaps the products of the next; all epilogue traffic
// moves through TMA boxes in shared memory.
#include <cuda.h>

#include <algorithm>

#include "context.cuh"
#include "step_tc.cuh"
#include "tc_ptx.cuh"

namespace fira {

namespace {

constexpr int BM = 128;           // tile rows = TMEM lanes
constexpr int BN_MAX = 256;       // tile columns = TMEM columns per accumulator
constexpr int BK = 64;            // k-block: 64 bf16 = 128 bytes
constexpr int A_STAGE_BYTES = BM * BK * 2;       // 16 KiB: 128 rows x 64 bf16
constexpr int CHUNK_BYTES = 64 * BK * 2;         // one 64 x 64 box: 8 KiB
constexpr int TMEM_COLS = 512;

struct TcMaps {
  CUtensorMap g1a;   // G, box for the projection product (2-D, or chunked 3-D: see encode_matrix_maps)
  CUtensorMap g1b;   // Pi [d][r] as chunks of 64 r: box of 64 r x 64 d x (BN / 128) chunks
  CUtensorMap g2a;   // back-projection A operand (Pi when left, X when right), box 64 x 128
  CUtensorMap g2b;   // back-projection B operand (X when left, Pi when right), box 64 x 128
  // boxes of the back-projection epilogue (64-byte swizzle)
  CUtensorMap eg;    // G [m][n] bf16, box 32 x 128
  CUtensorMap ew;    // W [m][n] bf16, box 32 x 128 (loaded and stored)
  // boxes of the projection epilogue
  CUtensorMap em;    // M [l][r] fp32, box 32 x 64, 128-byte swizzle (loaded and stored)
  CUtensorMap ev;    // V [l][r] fp32, same
  CUtensorMap en;    // N [l][r] bf16, box 32 x 64, 64-byte swizzle (stored)
  CUtensorMap er;    // R [l][r] bf16, same
  CUtensorMap ex;    // X [l][r] bf16, same (stored by the projection epilogue when it forms X itself)
};
static_assert(sizeof(TcMaps) % 64 == 0, "tensor maps must stay 64-byte aligned");

// r-extent of a projection tile; r is a multiple of 128 on this path
__device__ __forceinline__ int tile_bn(int r) { return (r % 256 == 0) ? 256 : 128; }

__device__ __forceinline__ uint4 pack8_bf16(const float (&v)[8]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
  __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]);
  __nv_bfloat162 d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 o;
  o.x = *reinterpret_cast<uint32_t*>(&a); o.y = *reinterpret_cast<uint32_t*>(&b);
  o.z = *reinterpret_cast<uint32_t*>(&c); o.w = *reinterpret_cast<uint32_t*>(&d);
  return o;
}
__device__ __forceinline__ void unpack8_bf16(const uint4& u, float (&v)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(p[i]);
    v[2 * i] = f.x; v[2 * i + 1] = f.y;
  }
}

#include "tc_project.cuh"
#include "tc_back_project.cuh"

// ============================================================================ small kernels
// w_j = 2 - ||pi_j||^2 for the columns of the stored projection [d][r]: 128 columns per block,
// two threads per column (even and odd rows), fp32 sums in a fixed order.
__global__ void __launch_bounds__(256)
k_tc_proj_weights(const MatDev* __restrict__ mats, const int* __restrict__ list, const int* __restrict__ wq_off,
                  const int* __restrict__ blk_start, int nlist, float* __restrict__ wq_all) {
  __shared__ float part[256];
  const int p = find_matrix(blk_start, nlist, blockIdx.x);
  const MatDev& mt = mats[list[p]];
  const int j = (blockIdx.x - blk_start[p]) * 128 + (threadIdx.x & 127);
  const int half = threadIdx.x >> 7;
  const __nv_bfloat16* P = static_cast<const __nv_bfloat16*>(mt.P);
  float acc = 0.f;
  if (j < mt.r)
    for (int i = half; i < mt.d; i += 2) {
      const float v = __bfloat162float(P[(long long)i * mt.r + j]);
      acc = fmaf(v, v, acc);
    }
  part[threadIdx.x] = acc;
  __syncthreads();
  if (half == 0 && j < mt.r) wq_all[wq_off[p] + j] = 2.f - (part[threadIdx.x] + part[threadIdx.x + 128]);
}

__global__ void __launch_bounds__(32)
k_tc_prep(const MatDev* __restrict__ mats, const int* __restrict__ list, int first, Hyper hp, float* __restrict__ fast) {
  const int p = first + blockIdx.x;            // one warp per matrix
  const MatDev& mt = mats[list[p]];
  if (threadIdx.x == 0) {
    const double s = (double)(mt.sc->t + 1);
    const float bias = (float)(sqrt(1.0 - pow((double)hp.beta2, s)) / (1.0 - pow((double)hp.beta1, s)));
    mt.sc->pad = bias;
    fast[2 * p] = bias;          // read by the projection epilogue
  }
  // the counters through which the projection epilogues of a row of tiles tell one another that
  // their partial sums are in place (behind the partial sums; see tc_colpart_floats)
  const int nparts = mt.r / tile_bn(mt.r);
  unsigned* cnt = reinterpret_cast<unsigned*>(mt.colpart + (long long)(3 + K1_GSQ_SPLIT) * nparts * mt.l);
  const int ncnt = 8 * ((mt.l + 2 * BM - 1) / (2 * BM));
  for (int i = threadIdx.x; i < ncnt; i += 32) cnt[i] = 0u;
}

// Copies between the caller's G and W and the copies with aligned rows, one block per row of a
// staged matrix.  dir 0: G -> Gs, W -> Ws; dir 1: Ws -> W.  The caller's rows start on 2-byte
// boundaries only; the copies' rows on 128-byte ones.  Both directions move 16-byte words on the
// aligned side and assemble them from (or cut them into) two neighbouring aligned words of the other
// side; a few elements at the ends of a row move one at a time.  No byte outside a row is written,
// and none outside [first row, last row] of either buffer is read.

// Bytes o .. o + 15 of the 32 bytes {a, b} (o even, 0 < o < 16).
__device__ __forceinline__ uint4 funnel16(const uint4 a, const uint4 b, int o) {
  const unsigned long long a0 = ((unsigned long long)a.y << 32) | a.x, a1 = ((unsigned long long)a.w << 32) | a.z;
  const unsigned long long b0 = ((unsigned long long)b.y << 32) | b.x, b1 = ((unsigned long long)b.w << 32) | b.z;
  unsigned long long lo, hi;
  if (o < 8) {
    const int sh = 8 * o;
    lo = (a0 >> sh) | (a1 << (64 - sh));
    hi = (a1 >> sh) | (b0 << (64 - sh));
  } else if (o == 8) {
    lo = a1; hi = b0;
  } else {
    const int sh = 8 * (o - 8);
    lo = (a1 >> sh) | (b0 << (64 - sh));
    hi = (b0 >> sh) | (b1 << (64 - sh));
  }
  return make_uint4((unsigned)lo, (unsigned)(lo >> 32), (unsigned)hi, (unsigned)(hi >> 32));
}

// Row of n elements from `src` (any 2-byte alignment) to `dst` (16-byte aligned).
__device__ __forceinline__ void copy_row_to_aligned(unsigned short* __restrict__ dst,
                                                    const unsigned short* __restrict__ src, int n, bool first_row) {
  const unsigned long long s = reinterpret_cast<unsigned long long>(src);
  const int o = (int)(s & 15);                                  // bytes past a 16-byte boundary
  const uint4* sw = reinterpret_cast<const uint4*>(s - o);
  uint4* dw = reinterpret_cast<uint4*>(dst);
  // words k < nw read sw[k], sw[k + 1]: bytes up to o + 2 n of the row; word 0 reaches o bytes back
  int nw = (o + 2 * n) / 16 - 1;
  if (nw < 0 || (o != 0 && first_row)) nw = 0;
  if (o == 0) {
    nw = n / 8;
#pragma unroll 4
    for (int k = threadIdx.x; k < nw; k += blockDim.x) dw[k] = sw[k];
  } else {
#pragma unroll 4
    for (int k = threadIdx.x; k < nw; k += blockDim.x) dw[k] = funnel16(sw[k], sw[k + 1], o);
  }
  for (int jj = 8 * nw + threadIdx.x; jj < n; jj += blockDim.x) dst[jj] = src[jj];
}

// Row of n elements from `src` (16-byte aligned, readable up to `pitch` elements) to `dst` (any alignment).
__device__ __forceinline__ void copy_row_from_aligned(unsigned short* __restrict__ dst,
                                                      const unsigned short* __restrict__ src, int n, int pitch) {
  const unsigned long long d = reinterpret_cast<unsigned long long>(dst);
  const int head = (int)(((16 - (d & 15)) & 15) / 2);           // elements before dst's first 16-byte boundary
  if (head >= n) { for (int jj = threadIdx.x; jj < n; jj += blockDim.x) dst[jj] = src[jj]; return; }
  uint4* dw = reinterpret_cast<uint4*>(dst + head);
  const uint4* sw = reinterpret_cast<const uint4*>(src);
  int nw = (n - head) / 8;                                      // whole aligned words of dst
  if (head == 0) {
#pragma unroll 4
    for (int k = threadIdx.x; k < nw; k += blockDim.x) dw[k] = sw[k];
  } else {
    nw = min(nw, pitch / 8 - 1);                                // word k reads sw[k] and sw[k + 1]
#pragma unroll 4
    for (int k = threadIdx.x; k < nw; k += blockDim.x) dw[k] = funnel16(sw[k], sw[k + 1], 2 * head);
  }
  for (int jj = threadIdx.x; jj < head; jj += blockDim.x) dst[jj] = src[jj];
  for (int jj = head + 8 * nw + threadIdx.x; jj < n; jj += blockDim.x) dst[jj] = src[jj];
}

__global__ void __launch_bounds__(256)
k_tc_stage(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
           const int* __restrict__ row_start, int first_row, int dir) {
  const int gr = blockIdx.x + first_row;
  const int p = find_matrix(row_start, nlist, gr);
  const MatDev& mt = mats[list[p]];
  const long long i = gr - row_start[p];
  const unsigned short* g = static_cast<const unsigned short*>(mt.G) + i * mt.ld;
  unsigned short* w = static_cast<unsigned short*>(mt.W) + i * mt.ld;
  unsigned short* gs = reinterpret_cast<unsigned short*>(mt.Gs) + i * mt.lds;
  unsigned short* ws = reinterpret_cast<unsigned short*>(mt.Ws) + i * mt.lds;
  if (dir == 0) {
    copy_row_to_aligned(gs, g, mt.n, i == 0);
    copy_row_to_aligned(ws, w, mt.n, i == 0);
  } else {
    copy_row_from_aligned(w, ws, mt.n, (int)mt.lds);
  }
}

// k_l and the partial sums of ||S||^2, 256 values of l per block.
__global__ void __launch_bounds__(256)
k_tc_colfactors(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
                const int* __restrict__ start, int first, Hyper hp) {
  __shared__ float red[8];
  const int gb = blockIdx.x + first;
  const int p = find_matrix(start, nlist, gb);
  const MatDev& mt = mats[list[p]];
  const int b = gb - start[p];
  const int l = b * 256 + threadIdx.x;
  float contrib = 0.f;
  if (l < mt.l) {
    const int nparts = mt.r / tile_bn(mt.r);
    float nn = 0.f, rn = 0.f, gs = 0.f;
    for (int q = 0; q < nparts; ++q) {
      nn += mt.colpart[(long long)(2 * q) * mt.l + l];
      rn += mt.colpart[(long long)(2 * q + 1) * mt.l + l];
    }
    for (int q = 2 * nparts; q < (2 + K1_GSQ_SPLIT) * nparts; ++q) gs += mt.colpart[(long long)q * mt.l + l];   // ||G_l||^2 in parts
    float rw = 0.f;                                      // sum_j (2 - ||pi_j||^2) R_lj^2
    for (int q = 0; q < nparts; ++q) rw += mt.colpart[(long long)((2 + K1_GSQ_SPLIT) * nparts + q) * mt.l + l];
    float k = sqrtf(nn) / (sqrtf(rn) + hp.eps);
    if (hp.mode & HYPER_MATRIX_SCALING) { mt.aux[l] = nn; mt.aux[mt.l + l] = rn; k = 1.f; }   // see k_finalize
    if (hp.mode & HYPER_NO_SCALING) k = 1.f;
    mt.kvec[l] = k;
    // only-scaling: S = G diag(k), so ||S_l||^2 = k_l^2 ||G_l||^2
    contrib = k * k * ((hp.mode & HYPER_ONLY_SCALING) ? gs : fmaxf(gs - rw, 0.f));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) contrib += __shfl_xor_sync(0xffffffffu, contrib, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = contrib;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += red[w];
    mt.part[b] = tot;
  }
}

// X = a_low N - a_res lambda k_l R in bf16, one warp per l.
__global__ void __launch_bounds__(256)
k_tc_form_x(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
            const int* __restrict__ row_start, int first_row, int rows_total, float a_low, float a_res,
            float* __restrict__ fast, int fused) {
  const int lane = threadIdx.x & 31;
  const int row = first_row + blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows_total) return;
  const int p = find_matrix(row_start, nlist, row);
  const MatDev& mt = mats[list[p]];
  const int l = row - row_start[p];
  const float lambda = mt.sc->lambda;
  if (fused && fuse_x_matrix(mt.d, mt.r)) return;      // k_tc_fix_x's matrix
  if (l == 0 && lane == 0) fast[2 * p + 1] = lambda;   // read by the back-projection epilogue
  const long long base = (long long)l * mt.r;
  const float c = a_res * lambda * mt.kvec[l];
  for (int j = lane * 8; j < mt.r; j += 256) {
    const uint4 nu = *reinterpret_cast<const uint4*>(mt.Nb + base + j);
    const uint4 ru = *reinterpret_cast<const uint4*>(mt.Rb + base + j);
    float nv[8], rv[8], x[8];
    unpack8_bf16(nu, nv);
    unpack8_bf16(ru, rv);
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = a_low * nv[e] - c * rv[e];
    *reinterpret_cast<uint4*>(mt.Xb + base + j) = pack8_bf16(x);
  }
}

// The matrices whose X the projection epilogue has formed for lambda = 1 (FUSE_X): where the limiter
// acted, X_lambda = a_low N - a_res lambda k_l R = lambda X + (1 - lambda) a_low N, with N rebuilt
// from the moments that the epilogue stored, by the epilogue's own arithmetic and rounded to bf16
// as it was there; the other matrices are left as they are.  blockIdx.y = matrix of the range, the
// blocks of a matrix stride over its rows, one warp per row.
__global__ void __launch_bounds__(256)
k_tc_fix_x(const MatDev* __restrict__ mats, const int* __restrict__ list, int first, float a_low, float eps,
           float* __restrict__ fast) {
  const int p = first + blockIdx.y;
  const MatDev& mt = mats[list[p]];
  if (!fuse_x_matrix(mt.d, mt.r)) return;              // k_tc_form_x's matrix
  const float lambda = mt.sc->lambda;
  if (blockIdx.x == 0 && threadIdx.x == 0) fast[2 * p + 1] = lambda;   // read by the back-projection epilogue
  if (lambda == 1.f) return;
  const int lane = threadIdx.x & 31;
  const float bias = fast[2 * p];                      // this step's bias factor (k_tc_prep)
  const float cn = (1.f - lambda) * a_low;
  for (int l = blockIdx.x * 8 + (threadIdx.x >> 5); l < mt.l; l += gridDim.x * 8) {
    const long long base = (long long)l * mt.r;
    for (int j = lane * 8; j < mt.r; j += 256) {
      const uint4 xu = *reinterpret_cast<const uint4*>(mt.Xb + base + j);
      const float4 m0 = *reinterpret_cast<const float4*>(mt.M + base + j), m1 = *reinterpret_cast<const float4*>(mt.M + base + j + 4);
      const float4 v0 = *reinterpret_cast<const float4*>(mt.V + base + j), v1 = *reinterpret_cast<const float4*>(mt.V + base + j + 4);
      const float mo[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
      const float vo[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      float xv[8], x[8];
      unpack8_bf16(xu, xv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float nv = __bfloat162float(__float2bfloat16_rn(__fdividef(bias * mo[e], fast_sqrt(vo[e]) + eps)));
        x[e] = lambda * xv[e] + cn * nv;
      }
      *reinterpret_cast<uint4*>(mt.Xb + base + j) = pack8_bf16(x);
    }
  }
}

// Self-test of the bounded waits: thread 0 waits on a barrier that nothing ever arrives on and gives
// up after `rounds` tries, raising the abort flag; a thread of the second warp sits in a wait with
// the ordinary limit, as the other roles of the product kernels do, and must leave when it sees the
// flag; a thread of the third warp polls a counter in global memory that nothing ever raises (the
// wait of the projection epilogues for the partial sums of their row of tiles) with the same small
// limit.  No copy is in flight and nothing else is touched.
__global__ void __launch_bounds__(96)
k_selftest_bounded_wait(unsigned* status, const uint32_t* never_raised, uint32_t rounds) {
  __shared__ uint64_t bars[2];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bars[0]), 1);
    ptx::mbar_init(ptx::smem_u32(&bars[1]), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  bool got = true;
  if (threadIdx.x == 0) got = ptx::mbar_wait(ptx::smem_u32(&bars[0]), 0, &abort_flag, rounds);
  if (threadIdx.x == 32) got = ptx::mbar_wait(ptx::smem_u32(&bars[1]), 0, &abort_flag);
  __shared__ int counter_gave_up;
  if (threadIdx.x == 64) counter_gave_up = ptx::wait_counter(never_raised, 0xffffffffu, &abort_flag, rounds) ? 0 : 1;
  __syncthreads();
  if (threadIdx.x == 0 && !got && abort_flag && counter_gave_up) atomicOr(status, DEV_STATUS_TIMEOUT);
}

// ============================================================================ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* sym = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(sym);
  return fn;
}

// bf16 row-major matrix [rows][cols] with leading dimension ld; box = box_c x box_r.
bool encode_map(CUtensorMap* out, const void* base, long long rows, long long cols, long long ld,
                int box_c, int box_r, int mode = 0) {
  // mode 0: bf16, 128-byte swizzle; 1: fp32, 128-byte swizzle; 2: bf16, 64-byte swizzle
  const bool fp32 = mode == 1;
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) { set_error("cuTensorMapEncodeTiled is not available"); return false; }
  const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t gstr[1] = {(cuuint64_t)ld * (fp32 ? 4 : 2)};
  const cuuint32_t box[2] = {(cuuint32_t)box_c, (cuuint32_t)box_r};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(out, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        mode == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed with code " + std::to_string((int)r)); return false; }
  return true;
}

// The same matrix seen as [cols / 64 chunks][rows][64]: one box brings `nchunk` adjacent
// 64-column chunks of box_r rows, each landing as its own swizzled 128-byte-row block (the
// layout of an MN-major operand).  Needs cols % 64 == 0: the chunk dimension has no ragged edge.
bool encode_map_chunked(CUtensorMap* out, const void* base, long long rows, long long cols, long long ld,
                        int box_r, int nchunk) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) { set_error("cuTensorMapEncodeTiled is not available"); return false; }
  const cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
  const cuuint64_t gstr[2] = {(cuuint64_t)ld * 2, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_r, (cuuint32_t)nchunk};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (chunked) failed with code " + std::to_string((int)r)); return false; }
  return true;
}

int host_tile_bn(int r) { return (r % 256 == 0) ? 256 : 128; }

}  // namespace

struct TcPlan {
  std::vector<TcMaps> maps;          // host image, one entry per matrix of the tc list
  TcMaps* maps_dev = nullptr;        // lives in the scratch buffer
  const int* list = nullptr;
  int nlist = 0;
  const int* k1_start = nullptr; int k1_tiles = 0;
  const int* k2_start = nullptr; int k2_tiles = 0;
  const int* col_start = nullptr; int col_blocks = 0;
  const int* row_start = nullptr; int rows_total = 0;
  const int* stage_list = nullptr; const int* stage_start = nullptr; int nstage = 0, stage_rows = 0;
  const int* npart = nullptr;
  ProjTileDesc* td1_dev = nullptr;   // per-tile records of the projection
  BackTileDesc* td2_dev = nullptr;   // per-tile records of the back-projection
  float* fast_dev = nullptr;         // per matrix of the list: {bias factor, lambda}
  float* wq_dev = nullptr;           // weights 2 - ||pi_j||^2 of all matrices of the list, r floats each
  const int* wq_off = nullptr;       // per matrix: its offset into wq_dev
  const int* wq_blk = nullptr;       // prefix sums of the blocks of k_tc_proj_weights
  int wq_blocks = 0;
  int num_sms = 148;
  int max_pairs_fused = 0;           // CTA pairs of the projection kernel that are resident at once (see launch_tc_step)
  bool attrs_set = false;
  // host copies of the prefix arrays (needed only to step a sub-range of the list)
  std::vector<int> h_k1, h_k2, h_cs, h_rs, h_sl, h_ss;
};

bool tc_supported(const fira_matrix_desc& d) {
  return d.dtype == FIRA_BF16 && d.r % 128 == 0 && d.m >= 256 && d.n >= 256;
}

bool tc_rows_aligned(const fira_matrix_desc& d) { return (d.ld ? d.ld : d.n) % 8 == 0; }

// TMA reads any width in place once the rows start on 16-byte boundaries (elements past the width
// come in as zeros), but it writes whole 16-byte units: a row whose width is not a multiple of 8
// elements gets up to 7 elements of its padding overwritten (with zeros).  Such matrices are worked
// on in place only if the caller has declared the padding writable; otherwise through the copies.
long long tc_staging_pitch(const fira_matrix_desc& d, uint32_t flags) {
  if (tc_rows_aligned(d) && (d.n % 8 == 0 || (flags & FIRA_FLAG_ROW_PADDING_WRITABLE))) return 0;
  return ((long long)d.n + 63) / 64 * 64;
}

size_t tc_colpart_floats(const fira_matrix_desc& d) {
  const size_t l = std::max(d.m, d.n);
  // N^2 and R^2 per r-tile, the partial G^2, the weighted R^2; then 8 counters per row of tiles
  // ([CTA rank][lane quarter]) for the exchange of the partial sums between the projection epilogues
  return (3 + K1_GSQ_SPLIT) * (size_t)(d.r / host_tile_bn(d.r)) * l + 8 * ((l + 2 * BM - 1) / (2 * BM));
}

size_t tc_part_floats(const fira_matrix_desc& d) { return ((size_t)std::max(d.m, d.n) + 255) / 256; }

static size_t proj_tiles(const fira_matrix_desc& d) {
  const int l = std::max(d.m, d.n);
  return (size_t)((l + 2 * BM - 1) / (2 * BM)) * (d.r / host_tile_bn(d.r));   // 256 l x BN r, one per CTA pair
}

static size_t back_tiles(const fira_matrix_desc& d) {
  return (size_t)((d.m + 2 * BM - 1) / (2 * BM)) * ((d.n + BN_MAX - 1) / BN_MAX);   // 256 x 256, one per CTA pair
}

// Device tables of this engine: tensor maps, fast scalars, back-projection tile records.
size_t tc_tables_bytes(const fira_hparams& hp, const fira_matrix_desc* descs, int count) {
  size_t ntc = 0, tiles2 = 0, tiles1 = 0, rsum = 0;
  for (int i = 0; i < count; ++i)
    if (engine_for(hp, descs[i]) == 1) { ++ntc; tiles2 += back_tiles(descs[i]); tiles1 += proj_tiles(descs[i]); rsum += descs[i].r; }
  return align_up(sizeof(TcMaps) * ntc) + align_up(2 * sizeof(float) * ntc) +
         align_up(sizeof(BackTileDesc) * tiles2) + align_up(sizeof(ProjTileDesc) * tiles1) + align_up(sizeof(float) * rsum);
}

static bool encode_matrix_maps(const MatDev& mt0, TcMaps& mp, bool only_g) {
  MatDev mt = mt0;
  if (mt.Gs) { mt.G = mt.Gs; mt.W = mt.Ws; mt.ld = mt.lds; }   // the kernels see the aligned copies
  // G is [m][n]: left -> 64 d rows of two 64-wide chunks of l (one chunked box when n % 64 == 0,
  // else two plain boxes); right -> box of 64 d x 128 l rows
  if (mt.left && mt.n % 64 == 0) {
    if (!encode_map_chunked(&mp.g1a, mt.G, mt.m, mt.n, mt.ld, 64, 2)) return false;
  } else if (!encode_map(&mp.g1a, mt.G, mt.m, mt.n, mt.ld, 64, mt.left ? 64 : 128)) return false;
  if (!encode_map(&mp.eg, mt.G, mt.m, mt.n, mt.ld, K2_ECOLS, 128, 2)) return false;
  if (!encode_map(&mp.ew, mt.W, mt.m, mt.n, mt.ld, K2_ECOLS, 128, 2)) return false;
  if (only_g) return true;
  if (!encode_map(&mp.em, mt.M, mt.l, mt.r, mt.r, K1_ECOLS, K1_EROWS, 1)) return false;
  if (!encode_map(&mp.ev, mt.V, mt.l, mt.r, mt.r, K1_ECOLS, K1_EROWS, 1)) return false;
  if (!encode_map(&mp.en, mt.Nb, mt.l, mt.r, mt.r, K1_ECOLS, K1_EROWS, 2)) return false;
  if (!encode_map(&mp.er, mt.Rb, mt.l, mt.r, mt.r, K1_ECOLS, K1_EROWS, 2)) return false;
  if (!encode_map(&mp.ex, mt.Xb, mt.l, mt.r, mt.r, K1_ECOLS, K1_EROWS, 2)) return false;
  if (!encode_map_chunked(&mp.g1b, mt.P, mt.d, mt.r, mt.r, 64, host_tile_bn(mt.r) / 128)) return false;
  const void* a2 = mt.left ? (const void*)mt.P : (const void*)mt.Xb;
  const void* b2 = mt.left ? (const void*)mt.Xb : (const void*)mt.P;
  const long long a2rows = mt.left ? mt.d : mt.l, b2rows = mt.left ? mt.l : mt.d;
  if (!encode_map(&mp.g2a, a2, a2rows, mt.r, mt.r, 64, 128)) return false;
  if (!encode_map(&mp.g2b, b2, b2rows, mt.r, mt.r, 64, 128)) return false;
  return true;
}

fira_status tc_build_plan(fira_ctx* c, std::vector<int>& ints) {
  if (c->tc_list.empty()) return FIRA_OK;
  TcPlan* pl = new TcPlan();
  c->tc = pl;
  cudaDeviceGetAttribute(&pl->num_sms, cudaDevAttrMultiProcessorCount, c->device);
  const std::vector<int>& lst = c->tc_list;
  std::vector<int> k1{0}, k2{0}, cs{0}, rs{0}, np, sl, ss{0}, wo, wb{0};
  int wsum = 0;
  for (int i : lst) {
    const MatDev& mt = c->mats[i];
    if (mt.Gs) { sl.push_back(i); ss.push_back(ss.back() + mt.m); }
    const int bn = host_tile_bn(mt.r);
    k1.push_back(k1.back() + ((mt.l + 2 * BM - 1) / (2 * BM)) * (mt.r / bn));
    k2.push_back(k2.back() + ((mt.m + 2 * BM - 1) / (2 * BM)) * ((mt.n + BN_MAX - 1) / BN_MAX));
    const int cb = (mt.l + 255) / 256;
    cs.push_back(cs.back() + cb);
    rs.push_back(rs.back() + mt.l);
    np.push_back(cb);
    wo.push_back(wsum); wsum += mt.r;
    wb.push_back(wb.back() + (mt.r + 127) / 128);
  }
  auto push_block = [&](const std::vector<int>& v) {
    size_t o = ints.size();
    ints.insert(ints.end(), v.begin(), v.end());
    return o;
  };
  const size_t o_list = push_block(lst), o_k1 = push_block(k1), o_k2 = push_block(k2),
               o_cs = push_block(cs), o_rs = push_block(rs), o_np = push_block(np),
               o_sl = push_block(sl), o_ss = push_block(ss), o_wo = push_block(wo), o_wb = push_block(wb);
  pl->wq_off = c->ints_dev + o_wo; pl->wq_blk = c->ints_dev + o_wb; pl->wq_blocks = wb.back();
  pl->list = c->ints_dev + o_list; pl->nlist = (int)lst.size();
  pl->k1_start = c->ints_dev + o_k1; pl->k1_tiles = k1.back();
  pl->k2_start = c->ints_dev + o_k2; pl->k2_tiles = k2.back();
  pl->col_start = c->ints_dev + o_cs; pl->col_blocks = cs.back();
  pl->row_start = c->ints_dev + o_rs; pl->rows_total = rs.back();
  pl->npart = c->ints_dev + o_np;
  pl->stage_list = c->ints_dev + o_sl; pl->stage_start = c->ints_dev + o_ss;
  pl->nstage = (int)sl.size(); pl->stage_rows = ss.back();
  pl->h_k1 = k1; pl->h_k2 = k2; pl->h_cs = cs; pl->h_rs = rs; pl->h_sl = sl; pl->h_ss = ss;
  pl->maps.resize(lst.size());
  char* tab = c->tc_maps_dev;
  pl->maps_dev = reinterpret_cast<TcMaps*>(tab); tab += align_up(sizeof(TcMaps) * lst.size());
  pl->fast_dev = reinterpret_cast<float*>(tab); tab += align_up(2 * sizeof(float) * lst.size());
  pl->td2_dev = reinterpret_cast<BackTileDesc*>(tab); tab += align_up(sizeof(BackTileDesc) * (size_t)pl->k2_tiles);
  pl->td1_dev = reinterpret_cast<ProjTileDesc*>(tab); tab += align_up(sizeof(ProjTileDesc) * (size_t)pl->k1_tiles);
  pl->wq_dev = reinterpret_cast<float*>(tab);
  {
    std::vector<BackTileDesc> td;
    td.reserve(pl->k2_tiles);
    for (size_t q = 0; q < lst.size(); ++q) {
      const MatDev& mt = c->mats[lst[q]];
      const int nrt = (mt.m + 2 * BM - 1) / (2 * BM), nct = (mt.n + BN_MAX - 1) / BN_MAX;
      for (int a = 0; a < nrt; ++a)
        for (int b = 0; b < nct; ++b) {
          BackTileDesc d;
          d.kvec = mt.kvec; d.slot = (int)q; d.i0 = a * 2 * BM; d.j0 = b * BN_MAX; d.nkb = mt.r / BK;
          d.n = mt.n; d.m_left = mt.m | (mt.left ? (int)0x80000000 : 0);
          td.push_back(d);
        }
    }
    if ((int)td.size() != pl->k2_tiles) { set_error("internal: tile count mismatch"); return FIRA_ERR_INVALID_ARG; }
    // projection tiles: the r-tiles of one l-range are neighbours, so that the CTA pairs
    // working on them share the G panel in L2
    std::vector<ProjTileDesc> tp;
    tp.reserve(pl->k1_tiles);
    for (size_t q = 0; q < lst.size(); ++q) {
      const MatDev& mt = c->mats[lst[q]];
      const int bn = host_tile_bn(mt.r), nrt = mt.r / bn, nlt = (mt.l + 2 * BM - 1) / (2 * BM);
      for (int a = 0; a < nlt; ++a)
        for (int b = 0; b < nrt; ++b) {
          ProjTileDesc d;
          d.colpart = mt.colpart; d.slot = (int)q; d.l0 = a * 2 * BM; d.r0 = b * bn;
          d.nkb = (mt.d + BK - 1) / BK; d.L = mt.l;
          d.bn_left = bn | ((mt.r / bn) << 16) | (mt.left ? (int)0x80000000 : 0) |
                      ((mt.left && mt.n % 64 == 0) ? PROJ_A_CHUNKED : 0) | (fuse_x_matrix(mt.d, mt.r) ? PROJ_FUSE_X : 0);
          tp.push_back(d);
        }
    }
    if ((int)tp.size() != pl->k1_tiles) { set_error("internal: tile count mismatch"); return FIRA_ERR_INVALID_ARG; }
    cudaError_t e = cudaMemcpyAsync(pl->td1_dev, tp.data(), sizeof(ProjTileDesc) * tp.size(),
                                    cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(pl->td2_dev, td.data(), sizeof(BackTileDesc) * td.size(),
                          cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // td dies at the end of this block
    if (e != cudaSuccess) { set_error(std::string("tile table upload: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  }
  // maps that do not depend on W / G; the G map is encoded when the pointers are known
  for (size_t q = 0; q < lst.size(); ++q) {
    MatDev mt = c->mats[lst[q]];
    mt.G = mt.P;   // placeholder addresses with valid alignment; replaced in tc_update_pointers
    mt.W = mt.P;
    if (!encode_matrix_maps(mt, pl->maps[q], false)) return FIRA_ERR_CUDA;
  }
  return FIRA_OK;
}

void tc_destroy_plan(fira_ctx* c) {
  delete c->tc;
  c->tc = nullptr;
}

fira_status tc_update_pointers(fira_ctx* c) {
  TcPlan* pl = c->tc;
  if (!pl) return FIRA_OK;
  for (size_t q = 0; q < c->tc_list.size(); ++q)
    if (!encode_matrix_maps(c->mats[c->tc_list[q]], pl->maps[q], true)) return FIRA_ERR_CUDA;
  cudaError_t e = cudaMemcpyAsync(pl->maps_dev, pl->maps.data(), sizeof(TcMaps) * pl->maps.size(),
                                  cudaMemcpyHostToDevice, c->stream);
  if (e != cudaSuccess) { set_error(std::string("tensor map upload: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  return FIRA_OK;
}

// ---------------------------------------------------------------- refresh products
static size_t gemm_job_tiles(const TcGemmJob& j) {
  const int L = j.mn_major ? j.n : j.m;
  return (size_t)((L + 2 * BM - 1) / (2 * BM)) * (j.r / host_tile_bn(j.r));
}

size_t tc_gemm_table_bytes(const TcGemmJob* jobs, int njobs) {
  size_t tiles = 0;
  for (int i = 0; i < njobs; ++i) tiles += gemm_job_tiles(jobs[i]);
  return align_up(sizeof(TcMaps) * (size_t)njobs) + align_up(sizeof(ProjTileDesc) * tiles);
}

fira_status tc_gemm_prepare(fira_ctx* c, const TcGemmJob* jobs, int njobs, char* table_dev, size_t table_bytes,
                            int* ntiles_out, cudaStream_t st) {
  if (tc_gemm_table_bytes(jobs, njobs) > table_bytes) { set_error("refresh: table area too small"); return FIRA_ERR_WORKSPACE_TOO_SMALL; }
  std::vector<TcMaps> maps((size_t)njobs);
  std::vector<ProjTileDesc> tiles;
  for (int q = 0; q < njobs; ++q) {
    const TcGemmJob& j = jobs[q];
    const int L = j.mn_major ? j.n : j.m, D = j.mn_major ? j.m : j.n;
    const int bn = host_tile_bn(j.r);
    const bool chunked = j.mn_major && j.n % 64 == 0;
    TcMaps& mp = maps[q];
    memset(&mp, 0, sizeof(mp));
    for (int part = 0; part < 2; ++part) {      // 0: the operands themselves, 1: their low parts (if any)
      const void* ga = part ? j.G_lo : j.G;
      const void* gb = part ? j.B_lo : j.B;
      CUtensorMap* ma = part ? &mp.g2a : &mp.g1a;
      CUtensorMap* mb = part ? &mp.g2b : &mp.g1b;
      if (ga) {
        if (chunked) {
          if (!encode_map_chunked(ma, ga, j.m, j.n, j.ld, 64, 2)) return FIRA_ERR_CUDA;
        } else if (!encode_map(ma, ga, j.m, j.n, j.ld, 64, j.mn_major ? 64 : 128)) return FIRA_ERR_CUDA;
      }
      if (gb && !encode_map_chunked(mb, gb, D, j.r, j.r, 64, bn / 128)) return FIRA_ERR_CUDA;
    }
    if (!encode_map(&mp.em, j.C, L, j.r, j.r, K1_ECOLS, K1_EROWS, 1)) return FIRA_ERR_CUDA;
    const int nseg = j.nseg > 1 ? j.nseg : 1;
    const int nkb_seg = (D + BK - 1) / BK;
    if (nseg > 3 || ((j.asel >> nseg) != 0) || ((j.bsel >> nseg) != 0) || (j.asel && !j.G_lo) || (j.bsel && !j.B_lo)) {
      set_error("internal: bad k-segments of a refresh product"); return FIRA_ERR_INVALID_ARG;
    }
    for (int l0 = 0; l0 < L; l0 += 2 * BM)
      for (int r0 = 0; r0 < j.r; r0 += bn) {
        ProjTileDesc d;
        d.colpart = reinterpret_cast<float*>(seg_word(nkb_seg, j.asel, j.bsel)); d.slot = q; d.l0 = l0; d.r0 = r0;
        d.nkb = nseg * nkb_seg; d.L = L;
        d.bn_left = bn | ((j.r / bn) << 16) | (j.mn_major ? (int)0x80000000 : 0) | (chunked ? PROJ_A_CHUNKED : 0);
        tiles.push_back(d);
      }
  }
  char* tiles_dev = table_dev + align_up(sizeof(TcMaps) * (size_t)njobs);
  cudaError_t e = cudaMemcpyAsync(table_dev, maps.data(), sizeof(TcMaps) * maps.size(), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(tiles_dev, tiles.data(), sizeof(ProjTileDesc) * tiles.size(), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) { set_error(std::string("refresh tables: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  *ntiles_out = (int)tiles.size();
  return FIRA_OK;
}

fira_status tc_gemm_run(fira_ctx* c, const char* table_dev, int njobs, int ntiles, cudaStream_t st) {
  // the shared-memory attribute of a kernel is a per-device setting
  static int sms_of_device[64] = {};
  if (c->device < 0 || c->device >= 64) { set_error("refresh product: device index out of range"); return FIRA_ERR_CUDA; }
  if (!sms_of_device[c->device]) {
    int n = 0;
    cudaError_t e = cudaFuncSetAttribute(k_tc_project<EPI_PLAIN, PSI_ADAM, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)K1_SMEM_BYTES);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess || n <= 0) { set_error(std::string("refresh product set-up: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
    sms_of_device[c->device] = n;
  }
  const int num_sms = sms_of_device[c->device];
  if (ntiles == 0) return FIRA_OK;
  const TcMaps* maps = reinterpret_cast<const TcMaps*>(table_dev);
  const ProjTileDesc* tiles = reinterpret_cast<const ProjTileDesc*>(table_dev + align_up(sizeof(TcMaps) * (size_t)njobs));
  Hyper hp{};
  k_tc_project<EPI_PLAIN, PSI_ADAM, 0><<<2 * std::min(ntiles, num_sms / 2), K1_THREADS, K1_SMEM_BYTES, st>>>(
      maps, tiles, ntiles, nullptr, nullptr, nullptr, hp, c->status_dev);
  return FIRA_OK;
}

fira_status tc_selftest_bounded_wait(fira_ctx* c, int rounds) {
  // the status word itself serves as the counter that never reaches its target
  k_selftest_bounded_wait<<<1, 96, 0, c->stream>>>(c->status_dev, c->status_dev, (uint32_t)rounds);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_error(std::string("bounded-wait self-test: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  return FIRA_OK;
}

int tc_phase_names(const char** out) {
  static const char* names[8] = {"k_tc_stage(in)", "k_tc_prep", "k_tc_project", "k_tc_colfactors",
                                 "k_finalize(tc)", "k_tc_form_x", "k_tc_back_project", "k_tc_stage(out)"};
  for (int i = 0; i < 8; ++i) out[i] = names[i];
  return 8;
}

int launch_tc_step(fira_ctx* c, const Hyper& hp, int qa, int qb) {
  TcPlan* pl = c->tc;
  if (!pl || pl->nlist == 0) return 0;
  cudaStream_t st = c->stream;
  if (!pl->attrs_set) {
    const void* k1s[4] = {(const void*)k_tc_project<EPI_ADAM, PSI_ADAM, 0>, (const void*)k_tc_project<EPI_ADAM, PSI_RMSPROP, 0>,
                          (const void*)k_tc_project<EPI_ADAM, PSI_ADAGRAD, 0>, (const void*)k_tc_project<EPI_ADAM, PSI_ADAM, 1>};
    const void* k1g[2] = {(const void*)k_tc_project<EPI_ADAM, PSI_ADAM, 0, 2>, (const void*)k_tc_project<EPI_ADAM, PSI_ADAM, 1, 2>};
    cudaError_t e1 = cudaSuccess;
    for (int i = 0; i < 4 && e1 == cudaSuccess; ++i)
      e1 = cudaFuncSetAttribute(k1s[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)K1_SMEM_BYTES);
    for (int i = 0; i < 2 && e1 == cudaSuccess; ++i)
      e1 = cudaFuncSetAttribute(k1g[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k1_smem_bytes(2));
    cudaError_t e2 = cudaFuncSetAttribute(k_tc_back_project<5, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k2_smem_bytes(5, 2));
    if (e2 == cudaSuccess)
      e2 = cudaFuncSetAttribute(k_tc_back_project<4, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)k2_smem_bytes(4, 3));
    if (e1 != cudaSuccess || e2 != cudaSuccess) {
      set_error(std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
      return -1;
    }
    // The epilogues of the fused projection kernel wait for one another across CTA pairs, so every
    // pair of its grid must be resident at once: the grid is capped at what the device can hold.
    {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(2 * (pl->num_sms / 2)); cfg.blockDim = dim3(K1_THREADS); cfg.dynamicSmemBytes = K1_SMEM_BYTES;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.attrs = at; cfg.numAttrs = 1;
      int nclusters = 0;
      const cudaError_t e3 = cudaOccupancyMaxActiveClusters(&nclusters, k1s[3], &cfg);
      if (e3 != cudaSuccess || nclusters <= 0) {
        set_error(std::string("cudaOccupancyMaxActiveClusters: ") + cudaGetErrorString(e3));
        return -1;
      }
      pl->max_pairs_fused = std::min(nclusters, pl->num_sms / 2);
      cfg.blockDim = dim3(k1_threads(2)); cfg.dynamicSmemBytes = k1_smem_bytes(2);
      const cudaError_t e4 = cudaOccupancyMaxActiveClusters(&nclusters, k1g[1], &cfg);
      if (e4 != cudaSuccess || nclusters <= 0) {
        set_error(std::string("cudaOccupancyMaxActiveClusters: ") + cudaGetErrorString(e4));
        return -1;
      }
      pl->max_pairs_fused = std::min(nclusters, pl->max_pairs_fused);
    }
    pl->attrs_set = true;
  }
  // the sub-range [qa, qb) of the list (qb < 0: all of it): first tile / block / row of every kernel
  // and their counts from the host copies of the prefix arrays
  if (qb < 0) { qa = 0; qb = pl->nlist; }
  if (qa >= qb) return 0;
  const int nq = qb - qa;
  const int k1a = pl->h_k1[qa], k1n = pl->h_k1[qb] - k1a;
  const int k2a = pl->h_k2[qa], k2n = pl->h_k2[qb] - k2a;
  const int csa = pl->h_cs[qa], csn = pl->h_cs[qb] - csa;
  const int rsa = pl->h_rs[qa], rsb = pl->h_rs[qb];
  // staged matrices (a subset of the list, both ascending) that fall into the range
  int sa = 0, sb = 0;
  for (int q = 0; q < pl->nstage; ++q) {
    if (pl->h_sl[q] < c->tc_list[qa]) ++sa;
    if (pl->h_sl[q] <= c->tc_list[qb - 1]) ++sb;
  }
  const int sra = pl->nstage ? pl->h_ss[sa] : 0, srn = pl->nstage ? pl->h_ss[sb] - sra : 0;
  PhaseTimer* tm = &c->timer;
  const MatDev* mats = c->mats_dev;
  if (c->proj_weights_dirty) {        // the stored projection has changed since the weights were taken
    k_tc_proj_weights<<<pl->wq_blocks, 256, 0, st>>>(mats, pl->list, pl->wq_off, pl->wq_blk, pl->nlist, pl->wq_dev);
    c->proj_weights_dirty = false;
  }
  if (srn) k_tc_stage<<<srn, 256, 0, st>>>(mats, pl->stage_list, pl->nstage, pl->stage_start, sra, 0);
  tm->mark(st);
  k_tc_prep<<<nq, 32, 0, st>>>(mats, pl->list, qa, hp, pl->fast_dev);
  tm->mark(st);
  // both tensor kernels: clusters of two CTAs, at most one CTA per SM
  // the plain step (Adam, column factors, residual kept) forms X in the projection epilogue
  const bool fused = (hp.mode & (HYPER_MATRIX_SCALING | HYPER_NO_SCALING | HYPER_NO_RESIDUAL | HYPER_ONLY_SCALING |
                                 HYPER_PSI_RMSPROP | HYPER_PSI_ADAGRAD)) == 0;
  const int k1_grid = 2 * std::min(k1n, fused ? pl->max_pairs_fused : pl->num_sms / 2);
  const ProjTileDesc* td1 = pl->td1_dev + k1a;
  int rmax = 0;
  for (int q = qa; q < qb; ++q) rmax = std::max(rmax, c->mats[c->tc_list[q]].r);
  // Short products are bound by the epilogue, which then runs with two groups of warps per CTA; long
  // ones (r = 1024 lists) are bound by the tensor pipe and keep one.
  const bool two_groups = rmax <= 512;
#define FIRA_LAUNCH_K1(PSI, FUSE)                                                     \
  k_tc_project<EPI_ADAM, PSI, FUSE><<<k1_grid, K1_THREADS, K1_SMEM_BYTES, st>>>(      \
      pl->maps_dev, td1, k1n, pl->fast_dev, pl->wq_dev, pl->wq_off, hp, c->status_dev)
  if (hp.mode & HYPER_PSI_RMSPROP) FIRA_LAUNCH_K1(PSI_RMSPROP, 0);
  else if (hp.mode & HYPER_PSI_ADAGRAD) FIRA_LAUNCH_K1(PSI_ADAGRAD, 0);
  else if (two_groups) {
    if (fused)
      k_tc_project<EPI_ADAM, PSI_ADAM, 1, 2><<<k1_grid, k1_threads(2), k1_smem_bytes(2), st>>>(
          pl->maps_dev, td1, k1n, pl->fast_dev, pl->wq_dev, pl->wq_off, hp, c->status_dev);
    else
      k_tc_project<EPI_ADAM, PSI_ADAM, 0, 2><<<k1_grid, k1_threads(2), k1_smem_bytes(2), st>>>(
          pl->maps_dev, td1, k1n, pl->fast_dev, pl->wq_dev, pl->wq_off, hp, c->status_dev);
  }
  else if (fused) FIRA_LAUNCH_K1(PSI_ADAM, 1);
  else FIRA_LAUNCH_K1(PSI_ADAM, 0);
#undef FIRA_LAUNCH_K1
  tm->mark(st);
  k_tc_colfactors<<<csn, 256, 0, st>>>(mats, pl->list, pl->nlist, pl->col_start, csa, hp);
  tm->mark(st);
  k_finalize<<<nq, 256, 0, st>>>(mats, pl->list + qa, nq, pl->npart + qa, hp, c->status_dev);
  tm->mark(st);
  if (hp.mode & HYPER_ONLY_SCALING) {
    // W <- W - lr phi(R) G: no back-projection; the element-wise update works on the caller's W and
    // G in place (whatever their pitch), so nothing is copied back from the aligned copies
    tm->mark(st);
    launch_scaled_gradient(mats, pl->list, pl->nlist, pl->k2_start, k2a, k2n, 2 * BM, 1, hp.lr, hp.a_res, st);
    tm->mark(st);
    tm->mark(st);
    return srn ? 6 : 5;
  }
  // X: the matrices whose projection epilogue formed it only need the limiter's correction
  bool any_fused = false, any_plain = false;
  for (int q = qa; q < qb; ++q) {
    const MatDev& mq = c->mats[c->tc_list[q]];
    if (fused && fuse_x_matrix(mq.d, mq.r)) any_fused = true; else any_plain = true;
  }
  if (any_plain)
    k_tc_form_x<<<(rsb - rsa + 7) / 8, 256, 0, st>>>(mats, pl->list, pl->nlist, pl->row_start, rsa, rsb,
                                                     hp.a_low, hp.a_res, pl->fast_dev, fused ? 1 : 0);
  if (any_fused) k_tc_fix_x<<<dim3(16, nq), 256, 0, st>>>(mats, pl->list, qa, hp.a_low, hp.eps, pl->fast_dev);
  tm->mark(st);
  // long products keep five operand stages; short ones trade one for more epilogue boxes in flight
  if (rmax >= 1024)
    k_tc_back_project<5, 2><<<2 * std::min(k2n, pl->num_sms / 2), K2_THREADS, k2_smem_bytes(5, 2), st>>>(
        pl->maps_dev, pl->td2_dev + k2a, k2n, pl->fast_dev, hp, c->status_dev);
  else
    k_tc_back_project<4, 3><<<2 * std::min(k2n, pl->num_sms / 2), K2_THREADS, k2_smem_bytes(4, 3), st>>>(
        pl->maps_dev, pl->td2_dev + k2a, k2n, pl->fast_dev, hp, c->status_dev);
  tm->mark(st);
  if (srn) k_tc_stage<<<srn, 256, 0, st>>>(mats, pl->stage_list, pl->nstage, pl->stage_start, sra, 1);
  tm->mark(st);
  return (srn ? 7 : 5) + (any_plain ? 1 : 0) + (any_fused ? 1 : 0);
}

}  // namespace fira
