// Projection product with Adam fused into its epilogue.  Included by step_tc.cu inside
// its namespace.
//
//   Rt[l][j] = sum_d G(d,l) Pi[d][j]          (R = P^T G, stored with the rank index contiguous)
//   M <- b1 M + (1-b1) R,  V <- b2 V + (1-b2) R^2,  N = bias M / (sqrt V + eps)     (Eq. 2-4)
//   writes M, V (fp32), N, R (bf16), the per-l partial sums ||N_l||^2, ||R_l||^2 and
//   sum_j w_j R_lj^2 with w_j = 2 - ||pi_j||^2 (pi_j = column j of the stored projection), and the
//   per-l sums ||G_l||^2: together they give ||S_l||^2 = ||G_l||^2 - sum_j w_j R_lj^2, which is
//   ||G_l - Pi R_l||^2 up to the off-diagonal part of Pi^T Pi - I
//
// CTA pairs (clusters of two, one CTA per SM) walk tiles of 256 l x BN r with
// tcgen05.mma.cta_group::2.  A = G: for m <= n an MN-major operand (G is [d][l], l
// contiguous: 64 d rows of two 64-wide chunks per CTA and stage), for m > n a K-major operand
// (one box of 64 d x 128 l).  B = Pi [d][r], MN-major; each CTA loads half of the tile's r range.
// No transposed copy of G or Pi is ever made, and no TMA multicast is used.
//
// One TMA instruction occupies the issuing thread for well over a hundred cycles, so a stage is
// loaded with two instructions: the chunks of an MN-major operand come as one 3-D box (the matrix
// seen as [chunk][row][64]).  Only a left-orientation G whose width is not a multiple of 64 falls
// back to one 2-D box per chunk.
//
// The epilogue moves M and V through shared memory with TMA in both directions (boxes of
// 64 rows x 32 columns, updated in place by one thread per row) and stores N and R the
// same way: ordinary global loads would be throttled by the few L1 lines that remain when
// nearly the whole L1/shared array is configured as shared memory.  The boxes of a tile come
// in the order (columns 0-31, rows 0-63), (columns 0-31, rows 64-127), (columns 32-63, ...):
// epilogue warps 0-1 take the even boxes, warps 2-3 the odd ones.  Five M/V buffers (an odd number,
// so that every buffer serves both row halves in turn) rotate over all boxes, so that loads run
// ahead; the N/R buffer of a box is the one of its row half.  Four operand stages and five M/V
// buffers share the shared memory: the step's time does not depend on the fifth stage (measured
// with 3 to 6 stages), while two more M/V boxes in flight raise the rate at which the epilogue
// streams M and V, which is what bounds the lists with a short product (350M: -7 %, 1B: -5 % on
// this kernel; 7B unchanged).
//
// ||G_l||^2: G passes through shared memory as the A operand anyway.  The r / BN tiles that share a
// panel of G split its k-blocks between them (tile `part` takes k-blocks part, part + r / BN, ...):
// eight more warps square and sum such an A stage while its MMAs run (the MMA issuer tells both CTAs
// when the stage has landed; the producer waits for the warps before it overwrites the stage, on
// those k-blocks only).  This replaces a separate pass over G in HBM.
//
// Warp roles: 0 operand producer (TMA); 1 MMA issuer (even CTA only) and TMEM owner;
// 2 epilogue loader (TMA); 3-6 epilogue; 7 one thread that stores the finished boxes;
// 8-15 sums of G^2; EG = 2: 16-19 a second group of epilogue warps.  A TMEM lane quarter belongs to
// the warps w with w % 4 equal to it, so the second group splits the columns, not the rows: both
// groups work on every box, each on 16 of its 32 columns, and the box barriers count both.  Lists
// whose products are short (r <= 512) are bound by this epilogue and take that instance.
//
// FUSE_X (the plain step: column factors, residual kept): the operand X = a_low N - a_res k_l R of the
// back-projection is formed here, for limiter factor 1, instead of in a pass of its own over N and R.
// k_l needs ||N_l|| and ||R_l|| over the whole rank range, i.e. over the r / BN tiles of a row of
// tiles, which different CTA pairs compute at about the same time.  So the epilogue makes two sweeps
// over its accumulator.  Sweep 1 does the moment update as before and puts the pair {bf16 N, bf16 R}
// back into each accumulator cell (tcgen05.st) instead of writing N and R out; it leaves its partial
// row sums in global memory and adds one to a counter of its (row of tiles, CTA rank, lane quarter).
// When the counter shows every tile of the row (a bounded poll: the pairs of a row run side by side,
// and a tile only ever waits for tiles whose index is at most three above its own, each of which
// follows, on its pair, a tile far below it, so the waits cannot form a cycle as long as every block
// of the grid is resident, which the launch ensures), the thread adds the partial sums in the fixed
// order that k_tc_colfactors uses, and sweep 2 reads the pairs back and writes X (through the map of
// the X buffer).  Nothing else leaves the kernel: where the limiter acts, k_tc_fix_x rebuilds N from
// the stored moments, X_lambda = lambda X + (1 - lambda) a_low N.  (Adam only: with RMSProp or Adagrad
// N cannot be rebuilt from V alone, and those steps keep the separate pass.)
constexpr int K1_STAGES = 4;
constexpr int K1_STAGE_BYTES = 2 * A_STAGE_BYTES;       // A: 128 l x 64 d, B half: 128 r x 64 d
constexpr int K1_ECOLS = 32;                            // columns per epilogue box
constexpr int K1_EROWS = 64;                            // rows per epilogue box
constexpr int K1_FBOX_BYTES = K1_EROWS * K1_ECOLS * 4;  // fp32 box: 8 KiB
constexpr int K1_HBOX_BYTES = K1_EROWS * K1_ECOLS * 2;  // bf16 box: 4 KiB
constexpr int K1_MVBUFS = 5;                            // {M box, V box}
constexpr int K1_NRBUFS = 2;                            // {N box, R box}, one per row half
constexpr int K1_MVBUF_BYTES = 2 * K1_FBOX_BYTES;
constexpr int K1_NRBUF_BYTES = 2 * K1_HBOX_BYTES;
constexpr int K1_BOX_THREADS = 64;                      // two warps work on a box
constexpr int K1_GSQ_WARPS = 8;
constexpr int K1_GSQ_SPLIT = K1_GSQ_WARPS / 2;          // partial sums of G^2 per tile and l
constexpr int K1_THREADS = 32 * (8 + K1_GSQ_WARPS);
// EG = 2: a second group of four epilogue warps (16-19).  The two groups work on the same boxes, each
// on one half of a box's 32 columns, and hand each other their halves of the row sums through XCH.
constexpr int K1_THREADS_EG2 = K1_THREADS + 128;
constexpr int K1_XCH_BYTES = BM * 4 * 4;                // per row: ||N||^2, ||R||^2, weighted ||R||^2 partials, k_l
constexpr size_t K1_SMEM_BYTES = (size_t)K1_STAGES * K1_STAGE_BYTES + (size_t)K1_MVBUFS * K1_MVBUF_BYTES +
                                 (size_t)K1_NRBUFS * K1_NRBUF_BYTES + 512;
static_assert(K1_SMEM_BYTES + K1_XCH_BYTES <= 227 * 1024, "shared memory budget");
constexpr int k1_threads(int eg) { return eg == 2 ? K1_THREADS_EG2 : K1_THREADS; }
constexpr size_t k1_smem_bytes(int eg) { return K1_SMEM_BYTES + (eg == 2 ? K1_XCH_BYTES : 0); }

// Per-tile record (256 l x BN r), built on the host once (32 bytes).
struct ProjTileDesc {
  float* colpart;      // partial sums of the tile's matrix: [2 part + which][l]; EPI_PLAIN: the k-segments
                       // of a split-precision product instead (see seg_word)
  int slot;            // index into the tensor-map table and the fast-scalar table
  int l0, r0;          // first unprojected index / first rank index of the tile
  int nkb;             // k-blocks: ceil(d / 64)
  int bn_left;         // bits 0-15: BN (128 or 256); 16-23: r / BN; 29: the epilogue forms X; 30: G comes as one chunked box; 31: left
  int L;               // number of unprojected indices of the matrix
};
static_assert(sizeof(ProjTileDesc) == 32, "ProjTileDesc layout");
constexpr int PROJ_A_CHUNKED = 1 << 30;
constexpr int PROJ_FUSE_X = 1 << 29;      // bn_left: this tile's epilogue forms X itself (FUSE_X kernels only)
// Which matrices take that route.  The second sweep lengthens the epilogue and the exchange makes the
// pairs of a row of tiles wait for the slowest of them.  Measured on the step: one r-tile per row (no
// exchange, 350M list, r = 256): -8 %; long products (7B list, d = 4096, four r-tiles): -6 to -7 %;
// short products with an exchange (1B list, d = 2048, two r-tiles): -2 % once the X boxes of the
// second sweep alternate between two buffers (+2 % before).  Shorter products with an exchange have
// not been measured and keep the separate pass.
constexpr int FUSE_X_MIN_D = 2048;
__host__ __device__ inline bool fuse_x_matrix(int d, int r) { return d >= FUSE_X_MIN_D || r <= 256; }

// EPI_PLAIN products may run over up to three k-segments that accumulate into the same tile: segment
// s multiplies A taken through the map g1a (bit s of asel clear) or g2a (set) with B taken through
// g1b or g2b (bsel), each over the same nkb_seg k-blocks.  With an fp32 matrix split into a bf16 high
// part and a bf16 remainder this gives hi*hi + hi*lo + lo*hi, a product good to about 2^-16.  The
// word travels in the record's pointer field: bits 0-31 nkb_seg (0: one segment over all k-blocks),
// 32-34 asel, 35-37 bsel.
__host__ __device__ inline unsigned long long seg_word(int nkb_seg, unsigned asel, unsigned bsel) {
  return (unsigned long long)(unsigned)nkb_seg | ((unsigned long long)(asel & 7u) << 32) | ((unsigned long long)(bsel & 7u) << 35);
}

struct ProjCtl {
  uint64_t full[K1_STAGES];     // (even CTA) both CTAs' operands of a stage have landed
  uint64_t empty[K1_STAGES];    // the MMAs reading a stage are done (both CTAs are told)
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];       // (even CTA) both CTAs' epilogues have drained an accumulator
  uint64_t afull[K1_STAGES];    // told by the MMA issuer to both CTAs: a stage that the G^2 warps read has landed
  uint64_t gdone[K1_STAGES];    // the G^2 warps have read that stage
  uint64_t efull[K1_MVBUFS][2]; // an M box and a V box have landed; one barrier per row half, so that
                                // its waiters (that half's warps) see every one of its phases
  uint64_t eready[K1_MVBUFS];   // the epilogue has finished M, V (in place) and N, R of a box
  uint64_t eempty[K1_MVBUFS];   // the stores have read M and V: the buffer is free
  uint64_t nrempty[K1_NRBUFS];  // the stores have read N and R: the buffer is free
  uint64_t xready[K1_NRBUFS][2];  // FUSE_X: a row half has finished an X box; X boxes alternate between the N
  uint64_t xempty[K1_NRBUFS][2];  //   and the R part of the half's buffer, each with its own pair of barriers
  uint64_t xsum[4];             // EG = 2, one per lane quarter: the second group's row sums are in XCH
  uint64_t xkl[4];              //   the first group has read them (and, FUSE_X, left k_l there)
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(ProjCtl) <= 512, "ProjCtl must fit its slot");

// sqrt.approx and the fast division are good to about 2 ulp each; N is rounded to bf16 next.
__device__ __forceinline__ float fast_sqrt(float x) {
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ ProjTileDesc load_desc(const ProjTileDesc* __restrict__ td, int t) {
  const int4 a = __ldg(reinterpret_cast<const int4*>(td + t));
  const int4 b = __ldg(reinterpret_cast<const int4*>(td + t) + 1);
  ProjTileDesc d;
  d.colpart = reinterpret_cast<float*>((static_cast<unsigned long long>(static_cast<unsigned>(a.y)) << 32) |
                                       static_cast<unsigned>(a.x));
  d.slot = a.z; d.l0 = a.w; d.r0 = b.x; d.nkb = b.y; d.bn_left = b.z; d.L = b.w;
  return d;
}

// EPI_ADAM: the step's kernel as described above.  EPI_PLAIN: the same product with the accumulator
// written out as it is, C[l][j] (fp32, through the `em` map): the products A^T Y and A Z of the
// projection refresh.  Then no M/V boxes are loaded, the output box of a row half is built in that
// half's N/R buffer, and the loader and the G^2 warps have nothing to do.
enum { EPI_ADAM = 0, EPI_PLAIN = 1 };
// PSI: the base optimizer of the EPI_ADAM epilogue (0 Adam, Eq. 2-4; 1 RMSProp; 2 Adagrad: M is then
// carried through unchanged).
enum { PSI_ADAM = 0, PSI_RMSPROP = 1, PSI_ADAGRAD = 2 };

template <int EPI, int PSI, int FUSE_X, int EG = 1>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(k1_threads(EG), 1)
k_tc_project(const TcMaps* __restrict__ maps, const ProjTileDesc* __restrict__ tdesc, int total_tiles,
             const float* __restrict__ fast, const float* __restrict__ wq_all, const int* __restrict__ wq_off,
             Hyper hp, unsigned* __restrict__ status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* tiles = smem_raw;
  unsigned char* mvbuf = tiles + (size_t)K1_STAGES * K1_STAGE_BYTES;
  unsigned char* nrbuf = mvbuf + (size_t)K1_MVBUFS * K1_MVBUF_BYTES;
  ProjCtl* ctl = reinterpret_cast<ProjCtl*>(nrbuf + (size_t)K1_NRBUFS * K1_NRBUF_BYTES);
  float4* xch = reinterpret_cast<float4*>(nrbuf + (size_t)K1_NRBUFS * K1_NRBUF_BYTES + 512);   // EG = 2 only
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();          // 0: issues the MMAs; 1: its partner
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  // the swizzled TMA tiles need a 1024-byte aligned base (same in both CTAs)
  const bool smem_ok = (ptx::smem_u32(smem_raw) & 1023u) == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < K1_STAGES; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->empty[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->afull[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->gdone[s]), K1_GSQ_WARPS);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_full[b]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->tmem_empty[b]), 2 * 4 * EG);   // every epilogue warp of the pair
    }
    for (int b = 0; b < K1_MVBUFS; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->efull[b][0]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->efull[b][1]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl->eready[b]), K1_BOX_THREADS * EG);
      ptx::mbar_init(ptx::smem_u32(&ctl->eempty[b]), 1);
    }
    for (int b = 0; b < K1_NRBUFS; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->nrempty[b]), 1);
      for (int x = 0; x < 2; ++x) {
        ptx::mbar_init(ptx::smem_u32(&ctl->xready[b][x]), K1_BOX_THREADS * EG);
        ptx::mbar_init(ptx::smem_u32(&ctl->xempty[b][x]), 1);
      }
    }
    for (int b = 0; b < 4; ++b) {
      ptx::mbar_init(ptx::smem_u32(&ctl->xsum[b]), 32);
      ptx::mbar_init(ptx::smem_u32(&ctl->xkl[b]), 32);
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
  const uint32_t mvbuf_u32 = ptx::smem_u32(mvbuf);
  const uint32_t nrbuf_u32 = ptx::smem_u32(nrbuf);

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer
    if (lane == 0 && smem_ok) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      uint32_t gmask = 0, gphase = 0;   // per stage: its occupant is read by the G^2 warps / parity of that wait
      ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const ProjTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int left = d.bn_left < 0;
        const int bn = d.bn_left & 0xffff;
        const int l0 = d.l0 + BM * (int)rank;             // this CTA's unprojected indices
        const int nparts = (d.bn_left >> 16) & 0xff;
        int gturn = EPI == EPI_ADAM ? d.r0 / bn : -1;     // next k-block that the G^2 warps read
        const uint32_t bytes = 2 * (A_STAGE_BYTES + (bn / 2) * BK * 2);   // both CTAs together
        const unsigned long long sw = EPI == EPI_PLAIN ? reinterpret_cast<unsigned long long>(d.colpart) : 0ull;
        const int nkb_seg = (int)(sw & 0xffffffffu) ? (int)(sw & 0xffffffffu) : d.nkb;
        const unsigned asel = (unsigned)(sw >> 32) & 7u, bsel = (unsigned)(sw >> 35) & 7u;
        const int rb0 = d.r0 + (bn / 2) * (int)rank;      // this CTA's half of the rank range
        int seg = 0, kk = 0;
        for (int kb = 0; kb < d.nkb; ++kb) {
          if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
          if ((gmask >> stage) & 1u) {                     // the previous occupant is still being squared
            if (!ptx::mbar_wait(ptx::smem_u32(&ctl->gdone[stage]), (gphase >> stage) & 1u, abort_flag)) { ok = false; break; }
            gphase ^= 1u << stage;
          }
          if (kb == gturn) { gturn += nparts; gmask |= 1u << stage; } else { gmask &= ~(1u << stage); }
          // all boxes of the pair complete on the even CTA's barrier
          const uint32_t fb = ptx::map_to_cta(ptx::smem_u32(&ctl->full[stage]), 0);
          const uint32_t sa = tiles_u32 + stage * K1_STAGE_BYTES;
          if (rank == 0) ptx::mbar_expect_tx(ptx::smem_u32(&ctl->full[stage]), bytes);
          const int k0 = kk * BK;
          const CUtensorMap* am = ((asel >> seg) & 1u) ? &mp->g2a : &mp->g1a;
          const CUtensorMap* bm = ((bsel >> seg) & 1u) ? &mp->g2b : &mp->g1b;
          if (++kk == nkb_seg) { kk = 0; ++seg; }
          if (d.bn_left & PROJ_A_CHUNKED) {
            ptx::tma_load_3d_pair(sa, am, fb, 0, k0, l0 >> 6);
          } else if (left) {
            ptx::tma_load_2d_pair(sa, am, fb, l0, k0);
            ptx::tma_load_2d_pair(sa + CHUNK_BYTES, am, fb, l0 + 64, k0);
          } else {
            ptx::tma_load_2d_pair(sa, am, fb, k0, l0);
          }
          ptx::tma_load_3d_pair(sa + A_STAGE_BYTES, bm, fb, 0, k0, rb0 >> 6);
          if (++stage == K1_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && rank == 0) {   // give copies in flight a bounded time to land
        for (int s = 0; s < K1_STAGES; ++s)
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (ptx::mbar_try_wait_cluster(ptx::smem_u32(&ctl->full[s]), (s < stage) ? phase : (phase ^ 1u))) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && smem_ok && rank == 0) {
      int stage = 0; uint32_t phase = 0; int buf = 0; uint32_t bphase = 0; bool ok = true;
      ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
      const uint32_t tmem = ctl->tmem_base;
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const ProjTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const int left = d.bn_left < 0;
        const int bn = d.bn_left & 0xffff;
        const uint32_t idesc = ptx::make_idesc_bf16(2 * BM, bn, left, 1);
        const int nparts = (d.bn_left >> 16) & 0xff;
        int gturn = EPI == EPI_ADAM ? d.r0 / bn : -1;     // next k-block that the G^2 warps read
        if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->tmem_empty[buf]), bphase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t dcol = tmem + buf * BN_MAX;
        for (int kb = 0; kb < d.nkb; ++kb) {
          if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->full[stage]), phase, abort_flag)) { ok = false; break; }
          if (kb == gturn) {                               // the G^2 warps may read this stage now
            gturn += nparts;
            ptx::mbar_arrive(ptx::smem_u32(&ctl->afull[stage]));     // (passed on to the odd CTA by a G^2 warp)
          }
          ptx::tc_fence_after();
          const uint32_t sa = tiles_u32 + stage * K1_STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            // MN-major: 16 k-rows of 128 bytes per step; K-major: 32 bytes along the row
            const uint64_t ad = left ? ptx::make_smem_desc(sa + k * 2048, CHUNK_BYTES, 1024)
                                     : ptx::make_smem_desc(sa + k * 32, 0, 1024);
            const uint64_t bd = ptx::make_smem_desc(sb + k * 2048, CHUNK_BYTES, 1024);
            ptx::umma_bf16_pair(dcol, ad, bd, idesc, (kb | k) ? 1u : 0u);
          }
          ptx::umma_commit_pair(ptx::smem_u32(&ctl->empty[stage]), 3);
          if (++stage == K1_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(ptx::smem_u32(&ctl->tmem_full[buf]), 3);
        if (++buf == 2) { buf = 0; bphase ^= 1u; }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ epilogue loader: M and V boxes
    if (EPI == EPI_ADAM && lane == 0 && smem_ok) {
      int mv = 0; uint32_t mvphase = 0; bool ok = true;
      ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const ProjTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int bn = d.bn_left & 0xffff;
        const int l0 = d.l0 + BM * (int)rank;
        for (int b = 0; b < 2 * (bn / K1_ECOLS); ++b) {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->eempty[mv]), mvphase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = ptx::smem_u32(&ctl->efull[mv][b & 1]);
          const uint32_t dst = mvbuf_u32 + mv * K1_MVBUF_BYTES;
          const int j = d.r0 + K1_ECOLS * (b >> 1), row = l0 + K1_EROWS * (b & 1);
          ptx::mbar_expect_tx(fb, K1_MVBUF_BYTES);
          ptx::tma_load_2d(dst, &mp->em, fb, j, row);
          ptx::tma_load_2d(dst + K1_FBOX_BYTES, &mp->ev, fb, j, row);
          if (++mv == K1_MVBUFS) { mv = 0; mvphase ^= 1u; }
        }
      }
    }
  } else if (warp >= 8 && warp < 8 + K1_GSQ_WARPS) {
    // ------------------------------------------------------------ sums of G^2 over the A stages
    if (EPI == EPI_ADAM && smem_ok) {
      const int w = warp - 8;
      const int kq = w >> 1;                             // left: d rows 16 kq .. + 15 of a stage
      int base = 0; uint32_t aphase = 0; bool ok = true;  // stage of the tile's first k-block; parities of afull
      ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const ProjTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const int left = d.bn_left < 0;
        const int bn = d.bn_left & 0xffff;
        const int nparts = (d.bn_left >> 16) & 0xff, part = d.r0 / bn;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int kb = part; kb < d.nkb; kb += nparts) {  // this tile's share of the panel's k-blocks
          const int stage = (base + kb) % K1_STAGES;
          // afull is used for these k-blocks only and every use is awaited here: its parity cannot alias
          if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->afull[stage]), (aphase >> stage) & 1u, abort_flag)) { ok = false; break; }
          aphase ^= 1u << stage;
          if (rank == 0 && w == 0 && lane == 0)            // a remote arrival would hold up the MMA issuer
            ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&ctl->afull[stage]), 1));
          {
            const unsigned char* sa = tiles + (size_t)stage * K1_STAGE_BYTES;
            if (left) {
              // chunk w % 2: [64 d rows][64 l], 128-byte rows, 16-byte slot ^= row % 8.
              // lane: slot lane % 8 (8 values of l), rows 16 kq + lane / 8, + 4, ...
              const unsigned char* ch = sa + (w & 1) * CHUNK_BYTES;
              const int slot = lane & 7;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int k = 16 * kq + (lane >> 3) + 4 * i;
                const uint4 u = *reinterpret_cast<const uint4*>(ch + k * 128 + ((slot ^ (k & 7)) << 4));
                float g[8];
                unpack8_bf16(u, g);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(g[e], g[e], acc[e]);
              }
            } else {
              // [128 l rows][64 d], 128-byte rows, slot ^= row % 8: half a row per thread
              const int row = 32 * (w & 3) + lane;
              const unsigned char* rp = sa + row * 128;
#pragma unroll
              for (int q = 4 * (w >> 2); q < 4 * (w >> 2) + 4; ++q) {
                const uint4 u = *reinterpret_cast<const uint4*>(rp + ((q ^ (row & 7)) << 4));
                float g[8];
                unpack8_bf16(u, g);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[0] = fmaf(g[e], g[e], acc[0]);
              }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctl->gdone[stage]));
          }
        }
        base = (base + d.nkb) % K1_STAGES;
        if (ok) {
          // slots after the 2 nparts partial sums of N^2 and R^2: [K1_GSQ_SPLIT part + quarter][l]
          float* gs = d.colpart + (long long)(2 * nparts + K1_GSQ_SPLIT * part) * d.L;
          const int lbase = d.l0 + BM * (int)rank;
          if (left) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 8);
              acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);
            }
            const int l = lbase + 64 * (w & 1) + 8 * lane;
            if (lane < 8 && l < d.L) {
              float* o = gs + (long long)kq * d.L + l;
              if ((d.L & 3) == 0 && l + 8 <= d.L) {      // rows of the table stay 16-byte aligned
                *reinterpret_cast<float4*>(o) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                *reinterpret_cast<float4*>(o + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) if (l + e < d.L) o[e] = acc[e];
              }
            }
          } else {
            const int l = lbase + 32 * (w & 3) + lane;   // slots 0 and 1: the two halves of the row; 2, 3: unused
            if (l < d.L) { gs[(long long)(w >> 2) * d.L + l] = acc[0]; gs[(long long)(2 + (w >> 2)) * d.L + l] = 0.f; }
          }
        }
      }
    }
  } else if (warp == 7) {
    // ------------------------------------------------------------ box storer
    if (lane == 0 && smem_ok) {
      int mv = 0; uint32_t mvphase = 0; bool ok = true;
      uint32_t xphase = 0;                                // FUSE_X: parities of xready, one bit per (row half, buffer part)
      ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
      for (int t = pair; t < total_tiles && ok; t += npairs) {
        const ProjTileDesc d = nd;
        if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
        const TcMaps* mp = &maps[d.slot];
        const int bn = d.bn_left & 0xffff;
        const int l0 = d.l0 + BM * (int)rank;
        const bool fuse = FUSE_X && (d.bn_left & PROJ_FUSE_X);
        for (int b = 0; b < 2 * (bn / K1_ECOLS); ++b) {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->eready[mv]), mvphase, abort_flag)) { ok = false; break; }
          const int nr = b & 1;
          const int j = d.r0 + K1_ECOLS * (b >> 1), row = l0 + K1_EROWS * nr;
          if (row < d.L) {
            const uint32_t src = mvbuf_u32 + mv * K1_MVBUF_BYTES, srn = nrbuf_u32 + nr * K1_NRBUF_BYTES;
            if (EPI == EPI_ADAM) {
              ptx::tma_store_2d(&mp->em, src, j, row);
              ptx::tma_store_2d(&mp->ev, src + K1_FBOX_BYTES, j, row);
              if (!fuse) {
                ptx::tma_store_2d(&mp->en, srn, j, row);
                ptx::tma_store_2d(&mp->er, srn + K1_HBOX_BYTES, j, row);
              }
            } else {
              ptx::tma_store_2d(&mp->em, srn, j, row);      // the fp32 output box sits in the N/R buffer
            }
            ptx::bulk_commit_group();
            ptx::bulk_wait_group_read<0>();              // the boxes have been read: the buffers are free
          }
          ptx::mbar_arrive(ptx::smem_u32(&ctl->eempty[mv]));
          if (!fuse) ptx::mbar_arrive(ptx::smem_u32(&ctl->nrempty[nr]));
          if (++mv == K1_MVBUFS) { mv = 0; mvphase ^= 1u; }
        }
        if (fuse && ok) {
          // second sweep of the epilogue: the X boxes of this tile, in the same order
          for (int b = 0; b < 2 * (bn / K1_ECOLS); ++b) {
            const int nr = b & 1, xs = (b >> 1) & 1, xbit = 2 * nr + xs;
            if (!ptx::mbar_wait(ptx::smem_u32(&ctl->xready[nr][xs]), (xphase >> xbit) & 1u, abort_flag)) { ok = false; break; }
            xphase ^= 1u << xbit;
            const int j = d.r0 + K1_ECOLS * (b >> 1), row = l0 + K1_EROWS * nr;
            if (row < d.L) {
              const uint32_t srn = nrbuf_u32 + nr * K1_NRBUF_BYTES + xs * K1_HBOX_BYTES;
              ptx::tma_store_2d(&mp->ex, srn, j, row);
              ptx::bulk_commit_group();
              ptx::bulk_wait_group_read<0>();
            }
            ptx::mbar_arrive(ptx::smem_u32(&ctl->xempty[nr][xs]));
          }
        }
      }
      ptx::bulk_wait_group_all();
    }
  } else if (smem_ok) {
    // ------------------------------------------------------------ epilogue: Adam on R
    constexpr int GC = K1_ECOLS / EG;                   // columns of a box that one group works on
    constexpr int QN = 4 / EG;                          //   in units of 8
    const int grp = (EG == 2 && warp >= 8) ? 1 : 0;     // group 1: warps 16-19
    const int q0 = QN * grp;
    uint32_t xphase = 0;                                // EG = 2: parity of xsum / xkl (one use per tile)
    const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
    const int row = quarter * 32 + lane;                // row of this CTA's half tile = TMEM lane
    const int half = quarter >> 1;                      // boxes with b % 2 == half are this warp's
    const int brow = row & (K1_EROWS - 1);              // row within the box
    const uint32_t frow = (uint32_t)brow * (K1_ECOLS * 4);  // fp32 boxes: 128-byte rows
    const uint32_t fsw = (uint32_t)brow & 7u;               //   128-byte swizzle: slot ^= row % 8
    const uint32_t hrow = (uint32_t)brow * (K1_ECOLS * 2);  // bf16 boxes: 64-byte rows
    const uint32_t hsw = (uint32_t)(brow >> 1) & 3u;        //   64-byte swizzle: slot ^= (row / 2) % 4
    const uint32_t tmem_empty0 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[0]), 0);
    const uint32_t tmem_empty1 = ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[1]), 0);
    int buf = 0; uint32_t bphase = 0;
    // This warp's boxes have the indices half, half + 2, ...: the M/V buffer is index % 3, and each
    // (buffer, half) barrier is used by every third of them.
    int mv = half; int mvuse = 0; uint32_t mvphase = 0;
    uint32_t nrphase = 0;                               // parity of this half's N/R buffer use
    uint32_t xeph = 0;                                  // FUSE_X: parities of this half's two X buffer parts
    const uint32_t nrempty = ptx::smem_u32(&ctl->nrempty[half]);
    unsigned char* nb = nrbuf + (size_t)half * K1_NRBUF_BYTES;
    unsigned char* rb = nb + K1_HBOX_BYTES;
    const uint32_t tmem = ctl->tmem_base;
    bool ok = true;
    ProjTileDesc nd = pair < total_tiles ? load_desc(tdesc, pair) : ProjTileDesc{};
    for (int t = pair; t < total_tiles && ok; t += npairs) {
      const ProjTileDesc d = nd;
      if (t + npairs < total_tiles) nd = load_desc(tdesc, t + npairs);
      const int bn = d.bn_left & 0xffff;
      const int l = d.l0 + BM * (int)rank + row;
      const float bias = EPI == EPI_ADAM ? fast[2 * d.slot] : 0.f;
      const float* wrow = EPI == EPI_ADAM ? wq_all + wq_off[d.slot] + d.r0 : nullptr;   // weights of this tile's rank range
      if (EPI == EPI_ADAM) asm volatile("prefetch.global.L1 [%0];" ::"l"(wrow));
      if (!ptx::mbar_wait_cluster(ptx::smem_u32(&ctl->tmem_full[buf]), bphase, abort_flag)) break;
      ptx::tc_fence_after();
      const uint32_t tcol = tmem + ((uint32_t)(quarter * 32) << 16) + buf * BN_MAX;
      const uint32_t te = buf ? tmem_empty1 : tmem_empty0;
      const int nch = bn / K1_ECOLS;
      const bool fuse = FUSE_X && (d.bn_left & PROJ_FUSE_X);
      float nn = 0.f, rn = 0.f, rw = 0.f;
      for (int c = 0; c < nch; ++c) {
        uint32_t rr[GC];
        __syncwarp();
        ptx::TmemCols<GC>::ld(tcol + K1_ECOLS * c + GC * grp, rr);
        // the next chunk's 32 weights (one 128-byte line) on their way into L1 meanwhile
        if (EPI == EPI_ADAM && c + 1 < nch)
          asm volatile("prefetch.global.L1 [%0];" ::"l"(wrow + K1_ECOLS * (c + 1)));
        ptx::tmem_ld_wait();
        if (!fuse && c == nch - 1) {                     // the accumulator has been read out
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(te);
        }
        if (EPI == EPI_ADAM && !ptx::mbar_wait(ptx::smem_u32(&ctl->efull[mv][half]), mvphase, abort_flag)) { ok = false; break; }
        if (!fuse && !ptx::mbar_wait(nrempty, nrphase ^ 1u, abort_flag)) { ok = false; break; }
        if (FUSE_X && !fuse && c == 0) {                 // the X boxes of an earlier tile have left the buffer too
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->xempty[half][0]), (xeph & 1u) ^ 1u, abort_flag) ||
              !ptx::mbar_wait(ptx::smem_u32(&ctl->xempty[half][1]), ((xeph >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        }
        unsigned char* mb = mvbuf + (size_t)mv * K1_MVBUF_BYTES;
        unsigned char* vb = mb + K1_FBOX_BYTES;
        if (EPI == EPI_PLAIN) {
          // 32 fp32 values of this row: eight 16-byte slots of a 128-byte row, slot ^= row % 8
#pragma unroll
          for (int qq = 0; qq < 8 / EG; ++qq) {
            const int q = qq + (8 / EG) * grp;
            *reinterpret_cast<uint4*>(nb + frow + (((uint32_t)q ^ fsw) << 4)) =
                make_uint4(rr[4 * qq], rr[4 * qq + 1], rr[4 * qq + 2], rr[4 * qq + 3]);
          }
        } else {
#pragma unroll
        for (int qq = 0; qq < QN; ++qq) {                // 8 columns at a time
          const int q = q0 + qq;
          const uint32_t f0 = frow + (((uint32_t)(2 * q) ^ fsw) << 4);
          const uint32_t f1 = frow + (((uint32_t)(2 * q + 1) ^ fsw) << 4);
          const float4 m0 = *reinterpret_cast<const float4*>(mb + f0);
          const float4 m1 = *reinterpret_cast<const float4*>(mb + f1);
          const float4 v0 = *reinterpret_cast<const float4*>(vb + f0);
          const float4 v1 = *reinterpret_cast<const float4*>(vb + f1);
          float mo[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
          float vo[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          const float4 w0 = __ldg(reinterpret_cast<const float4*>(wrow + K1_ECOLS * c + 8 * q));      // same for every lane
          const float4 w1 = __ldg(reinterpret_cast<const float4*>(wrow + K1_ECOLS * c + 8 * q + 4));
          const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
          float rv[8], nv[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            rv[e] = __uint_as_float(rr[8 * qq + e]);
            if (PSI == PSI_ADAM) {
              mo[e] = hp.beta1 * mo[e] + (1.f - hp.beta1) * rv[e];
              vo[e] = hp.beta2 * vo[e] + (1.f - hp.beta2) * rv[e] * rv[e];
              nv[e] = __fdividef(bias * mo[e], fast_sqrt(vo[e]) + hp.eps);
            } else {
              vo[e] = PSI == PSI_RMSPROP ? hp.beta2 * vo[e] + (1.f - hp.beta2) * rv[e] * rv[e] : vo[e] + rv[e] * rv[e];
              nv[e] = __fdividef(rv[e], fast_sqrt(vo[e]) + hp.eps);
            }
            nn = fmaf(nv[e], nv[e], nn);
            rn = fmaf(rv[e], rv[e], rn);
            rw = fmaf(wv[e] * rv[e], rv[e], rw);
          }
          *reinterpret_cast<float4*>(mb + f0) = make_float4(mo[0], mo[1], mo[2], mo[3]);
          *reinterpret_cast<float4*>(mb + f1) = make_float4(mo[4], mo[5], mo[6], mo[7]);
          *reinterpret_cast<float4*>(vb + f0) = make_float4(vo[0], vo[1], vo[2], vo[3]);
          *reinterpret_cast<float4*>(vb + f1) = make_float4(vo[4], vo[5], vo[6], vo[7]);
          if (fuse) {
            // the pair {bf16 N (low half), bf16 R (high half)} goes back into the accumulator cell
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const __nv_bfloat162 pr = __floats2bfloat162_rn(nv[e], rv[e]);
              rr[8 * qq + e] = *reinterpret_cast<const uint32_t*>(&pr);
            }
          } else {
            const uint32_t h = hrow + (((uint32_t)q ^ hsw) << 4);
            *reinterpret_cast<uint4*>(nb + h) = pack8_bf16(nv);
            *reinterpret_cast<uint4*>(rb + h) = pack8_bf16(rv);
          }
        }
        }
        if (fuse) {
          ptx::TmemCols<GC>::st(tcol + K1_ECOLS * c + GC * grp, rr);
          ptx::tmem_st_wait();
        }
        // hand the finished boxes to the storer: this thread's writes are visible to
        // the async proxy (TMA) before it arrives
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(ptx::smem_u32(&ctl->eready[mv]));
        if (!fuse) nrphase ^= 1u;
        mv += 2;                                         // this warp's next box is two further on
        if (mv >= K1_MVBUFS) mv -= K1_MVBUFS;
        if (++mvuse == K1_MVBUFS) { mvuse = 0; mvphase ^= 1u; }
      }
      if (EG == 2 && EPI == EPI_ADAM && ok) {
        // the second group hands its halves of the row sums to the first, which owns the row from here on
        if (grp == 1) {
          xch[row] = make_float4(nn, rn, rw, 0.f);
          ptx::mbar_arrive(ptx::smem_u32(&ctl->xsum[quarter]));
        } else {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->xsum[quarter]), xphase, abort_flag)) break;
          const float4 o = xch[row];
          nn += o.x; rn += o.y; rw += o.z;
        }
      }
      if (EPI == EPI_ADAM && ok && l < d.L && grp == 0) {
        // colpart[2 part][l] = partial ||N_l||^2, colpart[2 part + 1][l] = partial ||R_l||^2; after the
        // sums of G^2: colpart[(2 + K1_GSQ_SPLIT) nparts + part][l] = partial sum_j w_j R_lj^2
        const int part = d.r0 / bn, nparts = (d.bn_left >> 16) & 0xff;
        d.colpart[(long long)(2 * part) * d.L + l] = nn;
        d.colpart[(long long)(2 * part + 1) * d.L + l] = rn;
        d.colpart[(long long)((2 + K1_GSQ_SPLIT) * nparts + part) * d.L + l] = rw;
      }
      float kl = 0.f;
      if (fuse && ok && grp == 0) {
        // ---- the factor k_l of this thread's row, from the partial sums of every tile of the row of tiles
        const int nparts = (d.bn_left >> 16) & 0xff;
        float nt = 0.f, rt = 0.f;
        if (nparts > 1) {
          // counters behind the matrix's partial sums: [row of tiles][CTA rank][lane quarter]
          uint32_t* cnt = reinterpret_cast<uint32_t*>(d.colpart + (long long)(3 + K1_GSQ_SPLIT) * nparts * d.L) +
                          ((d.l0 / (2 * BM)) * 2 + (int)rank) * 4 + quarter;
          __threadfence();                               // this thread's partial sums, before the warp's count
          __syncwarp();
          int got = 1;
          if (lane == 0) {
            ptx::signal_counter(cnt);
            got = ptx::wait_counter(cnt, (uint32_t)nparts, abort_flag) ? 1 : 0;
          }
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) break;
          if (l < d.L) {
            for (int q = 0; q < nparts; ++q) {           // the order of k_tc_colfactors
              nt += __ldcg(d.colpart + (long long)(2 * q) * d.L + l);
              rt += __ldcg(d.colpart + (long long)(2 * q + 1) * d.L + l);
            }
          }
        } else {
          nt += nn; rt += rn;
        }
        kl = (l < d.L) ? sqrtf(nt) / (sqrtf(rt) + hp.eps) : 0.f;
      }
      if (EG == 2 && EPI == EPI_ADAM && ok) {
        // the first group has read the sums (XCH may be written again) and, FUSE_X, left k_l there
        if (grp == 0) {
          if (fuse) reinterpret_cast<float*>(&xch[row])[3] = kl;
          ptx::mbar_arrive(ptx::smem_u32(&ctl->xkl[quarter]));
        } else {
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->xkl[quarter]), xphase, abort_flag)) break;
          if (fuse) kl = reinterpret_cast<const float*>(&xch[row])[3];
        }
        xphase ^= 1u;
      }
      if (fuse && ok) {
        const float ck = hp.a_res * 1.0f * kl;           // k_tc_form_x's coefficient at lambda = 1
        // ---- sweep 2: X = a_low N - a_res k_l R as bf16 boxes
        for (int c = 0; c < nch; ++c) {
          uint32_t rr[GC];
          __syncwarp();
          ptx::TmemCols<GC>::ld(tcol + K1_ECOLS * c + GC * grp, rr);
          ptx::tmem_ld_wait();
          if (c == nch - 1) {                            // the accumulator has been read out
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(te);
          }
          const int xs = c & 1;                          // X boxes alternate between the two parts of the buffer
          if (!ptx::mbar_wait(ptx::smem_u32(&ctl->xempty[half][xs]), ((xeph >> xs) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          if (c == 0 && !ptx::mbar_wait(nrempty, nrphase ^ 1u, abort_flag)) { ok = false; break; }   // N, R of an earlier tile
          unsigned char* xb = nb + xs * K1_HBOX_BYTES;
#pragma unroll
          for (int qq = 0; qq < QN; ++qq) {
            const int q = q0 + qq;
            float xv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&rr[8 * qq + e]));
              xv[e] = hp.a_low * f.x - ck * f.y;
            }
            *reinterpret_cast<uint4*>(xb + hrow + (((uint32_t)q ^ hsw) << 4)) = pack8_bf16(xv);
          }
          ptx::fence_proxy_async_smem();
          ptx::mbar_arrive(ptx::smem_u32(&ctl->xready[half][xs]));
          xeph ^= 1u << xs;
        }
        if (!ok) break;
      }
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
