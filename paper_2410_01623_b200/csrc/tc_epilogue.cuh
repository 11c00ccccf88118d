// Epilogue building blocks of the tensor-core step kernels.  Included by step_tc.cu
// inside its namespace, after the tile constants.
//
// tcgen05.ld hands every thread one accumulator ROW (32 consecutive columns of its
// TMEM lane).  Touching global memory in that layout makes every warp instruction hit
// 32 different cache lines, which the load/store unit serialises.  So each epilogue
// warp first transposes its 32 x 32 fp32 chunk through a private shared-memory tile
// (rows of 128 bytes whose 16-byte slots are XOR-swizzled with the row number: both the
// row-wise writes and the reads below are free of bank conflicts) and then works in a
// COALESCED layout, in which the lanes of a warp cover
// a few whole rows of 64 or 128 contiguous bytes per instruction.
//
// Global operands that do not depend on the accumulators (M and V; G and W) are loaded
// one step ahead of the arithmetic into two alternating register buffers, across tile
// boundaries too, so that memory latency overlaps the TMEM reads, the arithmetic and
// the stores.

// Writes this thread's row (32 fp32 columns from TMEM) into the warp's staging tile.
__device__ __forceinline__ void stage_rows(float* stg, int lane, uint32_t taddr) {
  uint32_t rr[32];
  ptx::tmem_ld_32x32b_x32(taddr, rr);
  ptx::tmem_ld_wait();
  float4* row = reinterpret_cast<float4*>(stg + lane * STG_PITCH);
#pragma unroll
  for (int c = 0; c < 8; ++c)
    row[c ^ (lane & 7)] = make_float4(__uint_as_float(rr[4 * c]), __uint_as_float(rr[4 * c + 1]),
                         __uint_as_float(rr[4 * c + 2]), __uint_as_float(rr[4 * c + 3]));
  __syncwarp();
}

// ---------------------------------------------------------------------------- projection epilogue
// Coalesced layout of a 32-column fp32 chunk: lane -> row 4 i + lane / 8 (i = 0..7),
// columns 4 (lane % 8) .. + 3: eight lanes cover one 128-byte row segment of M or V.
// The unit of the register pipeline is half a chunk (i = 0..3 or 4..7).
struct ProjTile {
  float* M; float* V; __nv_bfloat16* Nb; __nv_bfloat16* Rb;   // at (row of i = 0, first column of this lane)
  float* colpart;
  float bias;
  int l0;          // unprojected index of the row of i = 0
  int L, r, nch, part, nparts;
  bool valid;
};

__device__ __forceinline__ ProjTile proj_tile(const MatDev* __restrict__ mats, const int* __restrict__ list,
                                              int nlist, const int* __restrict__ tile_start, int t,
                                              int total_tiles, int quarter, int half, int lane) {
  ProjTile pt;
  pt.valid = t < total_tiles;
  if (!pt.valid) { pt.L = 0; pt.l0 = 0; pt.nch = 0; return pt; }
  const int p = find_matrix(tile_start, nlist, t);
  const MatDev& mt = mats[list[p]];
  const int r = mt.r;
  const int bn = tile_bn(r), nrt = r / bn;
  const int local = t - tile_start[p];
  const int rt = local % nrt;
  pt.L = mt.l;
  pt.r = r;
  pt.l0 = (local / nrt) * BM + quarter * 32 + (lane >> 3);
  pt.nch = bn / 64;                         // chunks of 32 columns in this warp's half of the tile
  pt.nparts = 2 * nrt;
  pt.part = rt * 2 + half;
  pt.bias = mt.sc->pad;
  pt.colpart = mt.colpart;
  const long long off = (long long)pt.l0 * r + rt * bn + half * (bn / 2) + 4 * (lane & 7);
  pt.M = mt.M + off; pt.V = mt.V + off; pt.Nb = mt.Nb + off; pt.Rb = mt.Rb + off;
  return pt;
}

struct MVHalf { float4 m[4]; float4 v[4]; };

// item = 2 * chunk + half; rows 4 (4 half + ii) + lane / 8, ii = 0..3
__device__ __forceinline__ void load_mv(MVHalf& b, const ProjTile& pt, int item) {
  const int chunk = item >> 1, half = item & 1;
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    const int ro = 4 * (4 * half + ii);
    if (pt.l0 + ro < pt.L) {
      const long long off = (long long)ro * pt.r + 32 * chunk;
      b.m[ii] = *reinterpret_cast<const float4*>(pt.M + off);
      b.v[ii] = *reinterpret_cast<const float4*>(pt.V + off);
    }
  }
}

// Eq. 2-4 on half a chunk: R from the staging tile, M and V from the register buffer;
// writes M, V, and N, R as bf16; accumulates ||N||^2, ||R||^2 per row.
__device__ __forceinline__ void adam_half(const MVHalf& b, const ProjTile& pt, int item, const float* stg,
                                          int lane, const Hyper& hp, float (&nn)[8], float (&rn)[8]) {
  const int chunk = item >> 1, half = item & 1;
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    const int i = 4 * half + ii;
    const int ro = 4 * i;
    if (pt.l0 + ro < pt.L) {
      const int srow = ro + (lane >> 3);
      const float4 r4 = *reinterpret_cast<const float4*>(stg + srow * STG_PITCH + 4 * ((lane & 7) ^ (srow & 7)));
      const float rv[4] = {r4.x, r4.y, r4.z, r4.w};
      float mo[4] = {b.m[ii].x, b.m[ii].y, b.m[ii].z, b.m[ii].w};
      float vo[4] = {b.v[ii].x, b.v[ii].y, b.v[ii].z, b.v[ii].w};
      float nv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        mo[e] = hp.beta1 * mo[e] + (1.f - hp.beta1) * rv[e];
        vo[e] = hp.beta2 * vo[e] + (1.f - hp.beta2) * rv[e] * rv[e];
        nv[e] = pt.bias * mo[e] / (sqrtf(vo[e]) + hp.eps);
        nn[i] = fmaf(nv[e], nv[e], nn[i]);
        rn[i] = fmaf(rv[e], rv[e], rn[i]);
      }
      const long long off = (long long)ro * pt.r + 32 * chunk;
      *reinterpret_cast<float4*>(pt.M + off) = make_float4(mo[0], mo[1], mo[2], mo[3]);
      *reinterpret_cast<float4*>(pt.V + off) = make_float4(vo[0], vo[1], vo[2], vo[3]);
      __nv_bfloat162 n01 = __floats2bfloat162_rn(nv[0], nv[1]), n23 = __floats2bfloat162_rn(nv[2], nv[3]);
      __nv_bfloat162 r01 = __floats2bfloat162_rn(rv[0], rv[1]), r23 = __floats2bfloat162_rn(rv[2], rv[3]);
      uint2 nu, ru;
      nu.x = *reinterpret_cast<uint32_t*>(&n01); nu.y = *reinterpret_cast<uint32_t*>(&n23);
      ru.x = *reinterpret_cast<uint32_t*>(&r01); ru.y = *reinterpret_cast<uint32_t*>(&r23);
      *reinterpret_cast<uint2*>(pt.Nb + off) = nu;
      *reinterpret_cast<uint2*>(pt.Rb + off) = ru;
    }
  }
}
