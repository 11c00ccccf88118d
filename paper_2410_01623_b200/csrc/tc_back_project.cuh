// Back-projection product with the weight update fused into its epilogue.  Included
// by step_tc.cu inside its namespace.
//
//   D[i][j] = sum_q A(i,q) B(j,q) over the rank index q, both operands K-major:
//     left  (m <= n): A = Pi [d][r] (i = row of W), B = X [l][r] (j = column of W)
//     right (m >  n): A = X [l][r],                 B = Pi [d][r]
//   W[i][j] <- W[i][j] - lr (D[i][j] + a_res lambda k G[i][j]),  k per column (left) or row (right)
//
// One persistent CTA per SM walks 128 x 256 tiles of W.  All global traffic of the
// epilogue goes through TMA, because with nearly the whole L1/shared array configured
// as shared memory the few L1 lines left throttle ordinary loads: a loader thread
// brings 128 x 32 boxes of G and W into shared memory (64-byte swizzle, so a thread per
// row reads without bank conflicts), four epilogue warps combine them with the
// accumulator rows from tensor memory in place, and the W box is stored back by TMA.
//
// Warp roles: 0 operand producer (TMA), 1 MMA issuer (tcgen05) and TMEM owner,
// 2 epilogue loader (TMA), 3-6 epilogue.
constexpr int K2_STAGES = 3;
constexpr int K2_EBUFS = 4;
constexpr int K2_ECOLS = 32;                            // columns per epilogue box
constexpr int K2_EBOX_BYTES = BM * K2_ECOLS * 2;        // 8 KiB
constexpr int K2_EBUF_BYTES = 2 * K2_EBOX_BYTES;        // G box + W box
constexpr int K2_EPI_WARPS = 4;
constexpr int K2_EPI_THREADS = 32 * K2_EPI_WARPS;
constexpr int K2_THREADS = 32 * (3 + K2_EPI_WARPS);
constexpr int K2_NCH = BN_MAX / K2_ECOLS;               // 8 boxes per tile
constexpr size_t K2_SMEM_BYTES = (size_t)K2_STAGES * STAGE_BYTES + (size_t)K2_EBUFS * K2_EBUF_BYTES + 256 +
                                 2 * BN_MAX * sizeof(float);
static_assert(K2_SMEM_BYTES <= 227 * 1024, "shared memory budget");

// Per-tile record, built on the host once (32 bytes).
struct BackTileDesc {
  const float* kvec;   // factors k of the tile's matrix
  int slot;            // index into the tensor-map table and the fast-scalar table
  int i0, j0;          // first row / column of the tile in W
  int nkb;             // k-blocks: r / 64
  int n;               // columns of W
  int m_left;          // rows of W, bit 31 set for the left orientation
};
static_assert(sizeof(BackTileDesc) == 32, "BackTileDesc layout");

struct BackCtl {
  uint64_t full[K2_STAGES];
  uint64_t empty[K2_STAGES];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t efull[K2_EBUFS];
  uint64_t eempty[K2_EBUFS];
  uint64_t esync;        // the epilogue threads' own barrier
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(BackCtl) <= 256, "BackCtl must fit its slot");

__device__ __forceinline__ BackTileDesc load_desc(const BackTileDesc* __restrict__ td, int t) {
  const int4 a = __ldg(reinterpret_cast<const int4*>(td + t));
  const int4 b = __ldg(reinterpret_cast<const int4*>(td + t) + 1);
  BackTileDesc d;
  d.kvec = reinterpret_cast<const float*>((static_cast<unsigned long long>(static_cast<unsigned>(a.y)) << 32) |
                                          static_cast<unsigned>(a.x));
  d.slot = a.z; d.i0 = a.w; d.j0 = b.x; d.nkb = b.y; d.n = b.z; d.m_left = b.w;
  return d;
}

__global__ void __launch_bounds__(K2_THREADS, 1)
k_tc_back_project(const TcMaps* __restrict__ maps, const BackTileDesc* __restrict__ tdesc, int total_tiles,
                  const float* __restrict__ fast, Hyper hp, unsigned* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  if (ptx::smem_u32(smem_raw) & 1023u) {
    if (threadIdx.x == 0) atomicOr(status, DEV_STATUS_TIMEOUT);
    return;
  }
  unsigned char* tiles = smem_raw;
  unsigned char* ebuf = tiles + (size_t)K2_STAGES * STAGE_BYTES;
  BackCtl* ctl = reinterpret_cast<BackCtl*>(ebuf + (size_t)K2_EBUFS * K2_EBUF_BYTES);
  float* ksm = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(ctl) + 256);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < K2_STAGES; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_full[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_empty[b]), K2_EPI_WARPS);
    }
    for (int b = 0; b < K2_EBUFS; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->efull[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->eempty[b]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&ctl->esync), K2_EPI_THREADS);
    ctl->abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&ctl->tmem_base), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  volatile int* abort_flag = &ctl->abort_flag;
  const uint32_t tiles_u32 = ptx::smem_u32(tiles);
  const uint32_t ebuf_u32 = ptx::smem_u32(ebuf);

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      BackTileDesc nd = blockIdx.x < total_tiles ? load_desc(tdesc, blockIdx.x) : BackTileDesc{};
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const BackTileDesc d = nd;
        if (t + gridDim.x < total_tiles) nd = load_desc(tdesc, t + gridDim.x);
        const TcMaps* mp = &maps[d.slot];
        // the epilogue of this tile reads G and W; start moving them from HBM to L2 now
        for (int c = 0; c < BN_MAX / 64; ++c) {
          if (d.j0 + 64 * c < d.n) {
            ptx::tma_prefetch_l2_2d(&mp->pg, d.j0 + 64 * c, d.i0);
            ptx::tma_prefetch_l2_2d(&mp->pw, d.j0 + 64 * c, d.i0);
          }
        }
        for (int kb = 0; kb < d.nkb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = ptx::smem_u32(&ctl->full[stage]);
          const uint32_t sa = tiles_u32 + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
          ptx::mbar_expect_tx(fb, STAGE_BYTES);
          ptx::tma_load_2d(sa, &mp->g2a, fb, kb * BK, d.i0);
          ptx::tma_load_2d(sb, &mp->g2b, fb, kb * BK, d.j0);
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {   // give copies in flight a bounded time to land
        for (int s = 0; s < K2_STAGES; ++s)
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (ptx::mbar_try_wait(ptx::smem_u32(&ctl->full[s]), (s < stage) ? phase : (phase ^ 1u))) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; int buf = 0; uint32_t bphase = 0; bool ok = true;
      const uint32_t tmem = ctl->tmem_base;
      const uint32_t idesc = ptx::make_idesc_bf16(BM, BN_MAX, 0, 0);
      int nkb_next = blockIdx.x < total_tiles ? load_desc(tdesc, blockIdx.x).nkb : 0;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const int nkb = nkb_next;
        if (t + gridDim.x < total_tiles) nkb_next = load_desc(tdesc, t + gridDim.x).nkb;
        if (!ptx::mbar_wait(ptx::smem_u32(&ctl->tmem_empty[buf]), bphase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t dcol = tmem + buf * BN_MAX;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->full[stage]), phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = tiles_u32 + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t ad = ptx::make_smem_desc(sa + k * 32, 0, 1024);
            const uint64_t bd = ptx::make_smem_desc(sb + k * 32, 0, 1024);
            ptx::umma_bf16(dcol, ad, bd, idesc, (kb | k) ? 1u : 0u);
          }
          ptx::umma_commit(ptx::smem_u32(&ctl->empty[stage]));
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(ptx::smem_u32(&ctl->tmem_full[buf]));
        if (++buf == 2) { buf = 0; bphase ^= 1u; }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ epilogue loader
    if (lane == 0) {
      int eb = 0; uint32_t ephase = 0; bool ok = true;
      BackTileDesc nd = blockIdx.x < total_tiles ? load_desc(tdesc, blockIdx.x) : BackTileDesc{};
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const BackTileDesc d = nd;
        if (t + gridDim.x < total_tiles) nd = load_desc(tdesc, t + gridDim.x);
        const TcMaps* mp = &maps[d.slot];
        for (int c = 0; c < K2_NCH; ++c) {
          const int j = d.j0 + K2_ECOLS * c;
          if (j >= d.n) break;
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->eempty[eb]), ephase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = ptx::smem_u32(&ctl->efull[eb]);
          const uint32_t dst = ebuf_u32 + eb * K2_EBUF_BYTES;
          ptx::mbar_expect_tx(fb, K2_EBUF_BYTES);
          ptx::tma_load_2d(dst, &mp->eg, fb, j, d.i0);
          ptx::tma_load_2d(dst + K2_EBOX_BYTES, &mp->ew, fb, j, d.i0);
          if (++eb == K2_EBUFS) { eb = 0; ephase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;                // row of the tile = TMEM lane
    const int tid_e = threadIdx.x - 96;                 // 0..127 among the epilogue threads
    const uint32_t rowoff = (uint32_t)row * (K2_ECOLS * 2);
    const uint32_t sw = (uint32_t)(row >> 1) & 3u;      // 64-byte swizzle: slot ^= (row / 2) % 4
    const uint32_t esync = ptx::smem_u32(&ctl->esync);
    uint32_t sphase = 0;
    int buf = 0; uint32_t bphase = 0;
    int eb = 0; uint32_t ephase = 0;
    int prev_eb = -1;                                    // box whose store may still be reading
    int tile_parity = 0;
    const uint32_t tmem = ctl->tmem_base;
    bool ok = true;
    BackTileDesc nd = blockIdx.x < total_tiles ? load_desc(tdesc, blockIdx.x) : BackTileDesc{};
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      const BackTileDesc d = nd;
      if (t + gridDim.x < total_tiles) nd = load_desc(tdesc, t + gridDim.x);
      const int left = d.m_left < 0;
      const int m = d.m_left & 0x7fffffff;
      const float cres = hp.a_res * fast[2 * d.slot + 1];
      float* ks = ksm + tile_parity * BN_MAX;
      float krow = 0.f;
      if (left) {
        if (tid_e < BN_MAX / 4) {
          const int j = d.j0 + 4 * tid_e;               // n is a multiple of 8
          const float4 kv = (j < d.n) ? *reinterpret_cast<const float4*>(d.kvec + j) : make_float4(0.f, 0.f, 0.f, 0.f);
          *reinterpret_cast<float4*>(ks + 4 * tid_e) = kv;
        }
      } else if (d.i0 + row < m) {
        krow = d.kvec[d.i0 + row];
      }
      // all epilogue threads: the k values of this tile are in place
      ptx::mbar_arrive(esync);
      if (!ptx::mbar_wait(esync, sphase, abort_flag)) break;
      sphase ^= 1u;
      if (!ptx::mbar_wait(ptx::smem_u32(&ctl->tmem_full[buf]), bphase, abort_flag)) break;
      ptx::tc_fence_after();
      const uint32_t tcol = tmem + ((uint32_t)(quarter * 32) << 16) + buf * BN_MAX;
      const TcMaps* mp = &maps[d.slot];
      const int nch = min(K2_NCH, (d.n - d.j0 + K2_ECOLS - 1) / K2_ECOLS);
      for (int c = 0; c < nch; ++c) {
        uint32_t dd[32];
        __syncwarp();                                    // thread 0 may come late from its store
        ptx::tmem_ld_32x32b_x32(tcol + K2_ECOLS * c, dd);
        ptx::tmem_ld_wait();
        if (c == nch - 1) {                              // the accumulator has been read out
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->tmem_empty[buf]));
        }
        if (!ptx::mbar_wait(ptx::smem_u32(&ctl->efull[eb]), ephase, abort_flag)) { ok = false; break; }
        unsigned char* gb = ebuf + (size_t)eb * K2_EBUF_BYTES;
        unsigned char* wb = gb + K2_EBOX_BYTES;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t off = rowoff + (((uint32_t)q ^ sw) << 4);
          const uint4 gu = *reinterpret_cast<const uint4*>(gb + off);
          const uint4 wu = *reinterpret_cast<const uint4*>(wb + off);
          float g[8], w[8];
          unpack8_bf16(gu, g);
          unpack8_bf16(wu, w);
          if (left) {
            const float4 k0 = *reinterpret_cast<const float4*>(ks + K2_ECOLS * c + 8 * q);
            const float4 k1 = *reinterpret_cast<const float4*>(ks + K2_ECOLS * c + 8 * q + 4);
            const float kf[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = w[e] - hp.lr * (__uint_as_float(dd[8 * q + e]) + cres * kf[e] * g[e]);
          } else {
            const float ck = cres * krow;
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = w[e] - hp.lr * (__uint_as_float(dd[8 * q + e]) + ck * g[e]);
          }
          *reinterpret_cast<uint4*>(wb + off) = pack8_bf16(w);
        }
        // hand the finished W box to TMA: writes visible to the async proxy, then all
        // epilogue threads have arrived, then one thread stores
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(esync);
        if (!ptx::mbar_wait(esync, sphase, abort_flag)) { ok = false; break; }
        sphase ^= 1u;
        if (tid_e == 0) {
          ptx::tma_store_2d(&mp->ew, ptx::smem_u32(wb), d.j0 + K2_ECOLS * c, d.i0);
          ptx::bulk_commit_group();
          if (prev_eb >= 0) {
            // the store before this one has had a whole box time to read its source
            ptx::bulk_wait_group_read<1>();
            ptx::mbar_arrive(ptx::smem_u32(&ctl->eempty[prev_eb]));
          }
        }
        prev_eb = eb;
        if (++eb == K2_EBUFS) { eb = 0; ephase ^= 1u; }
      }
      tile_parity ^= 1;
      if (++buf == 2) { buf = 0; bphase ^= 1u; }
    }
    if (tid_e == 0) ptx::bulk_wait_group_all();          // shared memory must outlive the stores
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(ctl->tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && ctl->abort_flag) atomicOr(status, DEV_STATUS_TIMEOUT);
}
