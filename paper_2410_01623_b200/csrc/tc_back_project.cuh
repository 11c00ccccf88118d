// Back-projection product with the weight update fused into its epilogue.  Included
// by step_tc.cu inside its namespace.
//
//   D[i][j] = sum_q A(i,q) B(j,q) over the rank index q, both operands K-major:
//     left  (m <= n): A = Pi [d][r] (i = row of W), B = X [l][r] (j = column of W)
//     right (m >  n): A = X [l][r],                 B = Pi [d][r]
//   W[i][j] <- W[i][j] - lr (D[i][j] + a_res lambda k G[i][j]),  k per column (left) or row (right)
//
// CTA pairs (clusters of two, one CTA per SM) walk 256 x 256 tiles of W with
// tcgen05.mma.cta_group::2: each CTA owns 128 rows of the tile (its half of A, its
// accumulator rows in its own tensor memory) and loads only half of the B rows, which
// cuts the shared-memory footprint and the L2 -> SM traffic of the operands by a third.
// No TMA multicast is used: every CTA fetches its own boxes.
//
// All global traffic of the epilogue goes through TMA, because with nearly the whole
// L1/shared array configured as shared memory the few L1 lines left throttle ordinary
// loads: a loader thread brings 128 x 32 boxes of G and W into shared memory (64-byte
// swizzle, so a thread per row reads without bank conflicts), the epilogue warps combine
// them in place with the accumulator rows from tensor memory, and the W box is stored
// back by TMA.  Two groups of four epilogue warps take alternate boxes.
//
// Warp roles: 0 operand producer (TMA; the odd CTA's loads count on the even CTA's
// barrier, so that the MMA issuer waits on one barrier per stage); 1 MMA issuer (even
// CTA only) and TMEM owner; 2 epilogue loader (TMA); 3-10 epilogue; 11-12 one thread
// each that stores a group's finished W boxes (TMA) and hands the buffers back to the
// loader.  (Issuing the two boxes of a stage from two threads changed nothing: the
// stages wait for the data, not for the issuing thread.)
// Two splits of the shared memory between operand stages and epilogue boxes (template parameters
// of the kernel): 5 stages + 2 boxes in flight per epilogue group for long products (r >= 1024,
// tensor-bound), 4 stages + 3 boxes for short ones, whose tiles are bound by the rate at which the
// epilogue streams G and W (measured: 350M list -12 %, 1B list -6 % on this kernel with 4 + 3; the
// 7B list +3 % with it, so it keeps 5 + 2).
constexpr int K2_STAGE_BYTES = 2 * A_STAGE_BYTES;       // A: 128 x 64, B half: 128 x 64
constexpr int K2_GROUPS = 2;
constexpr int K2_ECOLS = 32;                            // columns per epilogue box
constexpr int K2_EBOX_BYTES = BM * K2_ECOLS * 2;        // 8 KiB
constexpr int K2_EBUF_BYTES = 2 * K2_EBOX_BYTES;        // G box + W box
constexpr int K2_GROUP_THREADS = 128;
constexpr int K2_THREADS = 32 * 3 + K2_GROUPS * K2_GROUP_THREADS + 32 * K2_GROUPS;
constexpr int K2_NCH = BN_MAX / K2_ECOLS;               // 8 boxes per tile
constexpr int K2_KS_GROUP = BN_MAX / K2_GROUPS;         // k values a group needs per tile (its own boxes)
constexpr int K2_KS_FLOATS = K2_GROUPS * 2 * K2_KS_GROUP;   // per group, two tile parities
constexpr size_t k2_smem_bytes(int stages, int gbufs) {
  return (size_t)stages * K2_STAGE_BYTES + (size_t)K2_GROUPS * gbufs * K2_EBUF_BYTES + 512 + K2_KS_FLOATS * sizeof(float);
}
static_assert(k2_smem_bytes(5, 2) <= 227 * 1024 && k2_smem_bytes(4, 3) <= 227 * 1024, "shared memory budget");

// Per-tile record (a 256 x 256 tile of W), built on the host once (32 bytes).
struct BackTileDesc {
  const float* kvec;   // factors k of the tile's matrix
  int slot;            // index into the tensor-map table and the fast-scalar table
  int i0, j0;          // first row / column of the tile in W
  int nkb;             // k-blocks: r / 64
  int n;               // columns of W
  int m_left;          // rows of W, bit 31 set for the left orientation
};
static_assert(sizeof(BackTileDesc) == 32, "BackTileDesc layout");

template <int K2_STAGES, int K2_GBUFS>
struct BackCtl {
  uint64_t full[K2_STAGES];     // (even CTA) both CTAs' operands of a stage have landed
  uint64_t empty[K2_STAGES];    // the MMAs reading a stage are done (both CTAs are told)
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];       // (even CTA) both CTAs' epilogues have drained an accumulator
  uint64_t efull[K2_GROUPS][K2_GBUFS];    // a G box and a W box have landed
  uint64_t eready[K2_GROUPS][K2_GBUFS];   // a group has finished a W box in place
  uint64_t eempty[K2_GROUPS][K2_GBUFS];   // its store has read the box: the buffer is free
  uint64_t esync[K2_GROUPS];    // each epilogue group's own barrier
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(BackCtl<5, 2>) <= 512 && sizeof(BackCtl<4, 3>) <= 512, "BackCtl must fit its slot");

__device__ __forceinline__ BackTileDesc load_desc(const BackTileDesc* __restrict__ td, int t) {
  const int4 a = __ldg(reinterpret_cast<const int4*>(td + t));
  const int4 b = __ldg(reinterpret_cast<const int4*>(td + t) + 1);
  BackTileDesc d;
  d.kvec = reinterpret_cast<const float*>((static_cast<unsigned long long>(static_cast<unsigned>(a.y)) << 32) |
                                          static_cast<unsigned>(a.x));
  d.slot = a.z; d.i0 = a.w; d.j0 = b.x; d.nkb = b.y; d.n = b.z; d.m_left = b.w;
  return d;
}

template <int K2_STAGES, int K2_GBUFS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(K2_THREADS, 1)
k_tc_back_project(const TcMaps* __restrict__ maps, const BackTileDesc* __restrict__ tdesc, int total_tiles,
                  const float* __restrict__ fast, Hyper hp, unsigned* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* tiles = smem_raw;
  unsigned char* ebuf = tiles + (size_t)K2_STAGES * K2_STAGE_BYTES;
  using Ctl = BackCtl<K2_STAGES, K2_GBUFS>;
  Ctl* ctl = reinterpret_cast<Ctl*>(ebuf + (size_t)K2_GROUPS * K2_GBUFS * K2_EBUF_BYTES);
  float* ksm = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(ctl) + 512);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();          // 0: issues the MMAs; 1: its partner
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  // the 128-byte swizzle of the TMA tiles needs a 1024-byte aligned base (same in both CTAs)
  const bool smem_ok = (ptx::smem_u32(smem_raw) & 1023u) == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < K2_STAGES; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_full[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_empty[b]), 2 * K2_GROUPS * 4);   // every epilogue warp of the pair
    }
    for (int g = 0; g < K2_GROUPS; ++g) {
      for (int b = 0; b < K2_GBUFS; ++b) {
        ptx::mbar_init(ptx::smem_u32(&ctl->efull[g][b]), 1);
        ptx::mbar_init(ptx::smem_u32(&ctl->eready[g][b]), K2_GROUP_THREADS);
        ptx::mbar_init(ptx::smem_u32(&ctl->eempty[g][b]), 1);
      }
      ptx::mbar_init(ptx::smem_u32(&ctl->esync[g]), K2_GROUP_THREADS);
    }
    ctl->abort_flag = smem_ok ? 0 : 1;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&ctl->tmem_base), TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();      // the partner's barriers exist before anything arrives on them
  ptx::tc_fence_after();
  volatile int* abort_flag = &ctl->abort_flag;
  const uint32_t tiles_u32 = ptx::smem_u32(tiles);
  const uint32_t ebuf_u32 = ptx::smem_u32(ebuf);

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer
    if (lane == 0 && smem_ok) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      BackTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : BackTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const BackTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int i0 = d.i0 + BM * (int)rank;            // this CTA's rows of W and of A
        const int jb0 = d.j0 + (BN_MAX / 2) * (int)rank; // this CTA's half of the B rows
        for (int kb = 0; kb < d.nkb; ++kb) {
          if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
          // all four boxes of the pair complete on the even CTA's barrier
          const uint32_t fb = ptx::map_to_cta(ptx::smem_u32(&ctl->full[stage]), 0);
          const uint32_t sa = tiles_u32 + stage * K2_STAGE_BYTES;
          if (rank == 0) ptx::mbar_expect_tx(ptx::smem_u32(&ctl->full[stage]), 2 * K2_STAGE_BYTES);
          ptx::tma_load_2d_pair(sa, &mp->g2a, fb, kb * BK, i0);
          ptx::tma_load_2d_pair(sa + A_STAGE_BYTES, &mp->g2b, fb, kb * BK, jb0);
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && rank == 0) {   // give copies in flight a bounded time to land
        for (int s = 0; s < K2_STAGES; ++s)
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (ptx::mbar_try_wait_cluster(ptx::smem_u32(&ctl->full[s]), (s < stage) ? phase : (phase ^ 1u))) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && smem_ok && rank == 0) {
      int stage = 0; uint32_t phase = 0; int buf = 0; uint32_t bphase = 0; bool ok = true;
      int nkb_next = pair < total_tiles ? load_desc(tdesc, pair).nkb : 0;
      const uint32_t tmem = ctl->tmem_base;
      const uint32_t idesc = ptx::make_idesc_bf16(2 * BM, BN_MAX, 0, 0);
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const int nkb = nkb_next;
        if (t + npairs < total_tiles) nkb_next = load_desc(tdesc, t + npairs).nkb;
        if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->tmem_empty[buf]), bphase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t dcol = tmem + buf * BN_MAX;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->full[stage]), phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = tiles_u32 + stage * K2_STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t ad = ptx::make_smem_desc(sa + k * 32, 0, 1024);
            const uint64_t bd = ptx::make_smem_desc(sb + k * 32, 0, 1024);
            ptx::umma_bf16_pair(dcol, ad, bd, idesc, (kb | k) ? 1u : 0u);
          }
          ptx::umma_commit_pair(ptx::smem_u32(&ctl->empty[stage]), 3);
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(ptx::smem_u32(&ctl->tmem_full[buf]), 3);
        if (++buf == 2) { buf = 0; bphase ^= 1u; }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ epilogue loader
    if (lane == 0 && smem_ok) {
      int eb[K2_GROUPS] = {0, 0}; uint32_t ephase[K2_GROUPS] = {0, 0}; bool ok = true;
      BackTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : BackTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const BackTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int i0 = d.i0 + BM * (int)rank;
        for (int c = 0; c < K2_NCH; ++c) {
          const int j = d.j0 + K2_ECOLS * c;
          if (j >= d.n) break;
          const int g = c & 1;
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->eempty[g][eb[g]]), ephase[g] ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = ptx::smem_u32(&ctl->efull[g][eb[g]]);
          const uint32_t dst = ebuf_u32 + (g * K2_GBUFS + eb[g]) * K2_EBUF_BYTES;
          ptx::mbar_expect_tx(fb, K2_EBUF_BYTES);
          ptx::tma_load_2d(dst, &mp->eg, fb, j, i0);
          ptx::tma_load_2d(dst + K2_EBOX_BYTES, &mp->ew, fb, j, i0);
          if (++eb[g] == K2_GBUFS) { eb[g] = 0; ephase[g] ^= 1u; }
        }
      }
    }
  } else if (warp >= 3 + 4 * K2_GROUPS) {
    // ------------------------------------------------------------ W box storer of one group
    if (lane == 0 && smem_ok) {
      const int g = warp - (3 + 4 * K2_GROUPS);
      int eb = 0; uint32_t rphase = 0; bool ok = true;
      BackTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : BackTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const BackTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int i0 = d.i0 + BM * (int)rank;
        const int m = d.m_left & 0x7fffffff;
        const int nch = min(K2_NCH, (d.n - d.j0 + K2_ECOLS - 1) / K2_ECOLS);
        for (int c = g; c < nch; c += K2_GROUPS) {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->eready[g][eb]), rphase, abort_flag)) { ok = false; break; }
          if (i0 < m) {
            ptx::tma_store_2d(&mp->ew, ebuf_u32 + (g * K2_GBUFS + eb) * K2_EBUF_BYTES + K2_EBOX_BYTES,
                              d.j0 + K2_ECOLS * c, i0);
            ptx::bulk_commit_group();
            ptx::bulk_wait_group_read<0>();              // the box has been read: the buffer is free
          }
          ptx::mbar_arrive(ptx::smem_u32(&ctl->eempty[g][eb]));
          if (++eb == K2_GBUFS) { eb = 0; rphase ^= 1u; }
        }
      }
      ptx::bulk_wait_group_all();
    }
  } else if (smem_ok) {
    // ------------------------------------------------------------ epilogue
    const int ew = warp - 3;
    const int g = ew >> 2;                               // group: boxes g, g + 2, g + 4, g + 6
    const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;                // row of this CTA's half tile = TMEM lane
    const int tid_g = (ew & 3) * 32 + lane;             // 0..127 within the group
    const uint32_t rowoff = (uint32_t)row * (K2_ECOLS * 2);
    const uint32_t sw = (uint32_t)(row >> 1) & 3u;      // 64-byte swizzle: slot ^= (row / 2) % 4
    const uint32_t esync = ptx::smem_u32(&ctl->esync[g]);
    const uint32_t tmem_empty0 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[0]), 0);
    const uint32_t tmem_empty1 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[1]), 0);
    uint32_t sphase = 0;
    int buf = 0; uint32_t bphase = 0;
    int eb = 0; uint32_t ephase = 0;
    int tile_parity = 0;
    const uint32_t tmem = ctl->tmem_base;
    bool ok = true;
    BackTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : BackTileDesc{};
    for (int t = pair; t < total_tiles && ok; t += npairs) {
      const BackTileDesc d = nd;
      if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
      const int left = d.m_left < 0;
      const int m = d.m_left & 0x7fffffff;
      const int i0 = d.i0 + BM * (int)rank;
      const float cres = hp.a_res * fast[2 * d.slot + 1];
      float* ks = ksm + (g * 2 + tile_parity) * K2_KS_GROUP;   // box c of this group at ks + 32 (c / 2)
      float krow = 0.f;
      if (left) {
        if (tid_g < K2_KS_GROUP / 4) {
          const int box = K2_GROUPS * (tid_g >> 3) + g;  // 8 float4 per box of 32 columns
          const int j = d.j0 + K2_ECOLS * box + 4 * (tid_g & 7);   // (the k table is padded to 64 floats)
          const float4 kv = (j < d.n) ? *reinterpret_cast<const float4*>(d.kvec + j) : make_float4(0.f, 0.f, 0.f, 0.f);
          *reinterpret_cast<float4*>(ks + 4 * tid_g) = kv;
        }
      } else if (i0 + row < m) {
        krow = d.kvec[i0 + row];
      }
      // all threads of the group: the k values of this tile are in place
      ptx::mbar_arrive(esync);
      if (!ptx::mbar_wait(esync, sphase, abort_flag)) break;
      sphase ^= 1u;
      if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->tmem_full[buf]), bphase, abort_flag)) break;
      ptx::tc_fence_after();
      const uint32_t tcol = tmem + ((uint32_t)(quarter * 32) << 16) + buf * BN_MAX;
      const int nch = min(K2_NCH, (d.n - d.j0 + K2_ECOLS - 1) / K2_ECOLS);
      const uint32_t te = buf ? tmem_empty1 : tmem_empty0;
      if (g >= nch) {                                    // this group has no box in this tile
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(te);
      }
      for (int c = g; c < nch; c += K2_GROUPS) {
        uint32_t dd[32];
        __syncwarp();
        ptx::tmem_ld_32x32b_x32(tcol + K2_ECOLS * c, dd);
        ptx::tmem_ld_wait();
        if (c + K2_GROUPS >= nch) {                      // this warp has read all it needs of the accumulator
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(te);
        }
        if (!ptx::mbar_wait(ptx::smem_u32(&ctl->efull[g][eb]), ephase, abort_flag)) { ok = false; break; }
        unsigned char* gb = ebuf + (size_t)(g * K2_GBUFS + eb) * K2_EBUF_BYTES;
        unsigned char* wb = gb + K2_EBOX_BYTES;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t off = rowoff + (((uint32_t)q ^ sw) << 4);
          const uint4 gu = *reinterpret_cast<const uint4*>(gb + off);
          const uint4 wu = *reinterpret_cast<const uint4*>(wb + off);
          float gg[8], w[8];
          unpack8_bf16(gu, gg);
          unpack8_bf16(wu, w);
          if (left) {
            const float4 k0 = *reinterpret_cast<const float4*>(ks + K2_ECOLS * (c / K2_GROUPS) + 8 * q);
            const float4 k1 = *reinterpret_cast<const float4*>(ks + K2_ECOLS * (c / K2_GROUPS) + 8 * q + 4);
            const float kf[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = w[e] - hp.lr * (__uint_as_float(dd[8 * q + e]) + cres * kf[e] * gg[e]);
          } else {
            const float ck = cres * krow;
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = w[e] - hp.lr * (__uint_as_float(dd[8 * q + e]) + ck * gg[e]);
          }
          *reinterpret_cast<uint4*>(wb + off) = pack8_bf16(w);
        }
        // hand the finished W box to the storer: this thread's writes are visible to
        // the async proxy (TMA) before it arrives
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(ptx::smem_u32(&ctl->eready[g][eb]));
        if (++eb == K2_GBUFS) { eb = 0; ephase ^= 1u; }
      }
      tile_parity ^= 1;
      if (++buf == 2) { buf = 0; bphase ^= 1u; }
    }
  }
  // Neither CTA may leave while its partner can still reach into its shared memory
  // (operand reads by the MMAs, barrier arrivals).
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(ctl->tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && ctl->abort_flag) atomicOr(status, DEV_STATUS_TIMEOUT);
}
