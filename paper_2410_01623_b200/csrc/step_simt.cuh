// Launch interface of the grouped fp32 CUDA-core step kernels.
#pragma once
#include "common.cuh"

namespace fira {

// Device-resident schedule of one list of matrices.  `list` holds indices into
// `mats`; the *_start arrays have nlist + 1 ascending entries (prefix sums).
struct SimtPlan {
  const MatDev* mats = nullptr;
  const int* list = nullptr;
  int nlist = 0;
  const int* proj_tile_start = nullptr;  // 64 x 64 tiles of Rt (l x r)
  int proj_tiles = 0;
  const int* row_start = nullptr;        // rows l
  int rows_total = 0;
  const int* w_tile_start = nullptr;     // 64 x 64 tiles of W (m x n)
  int w_tiles = 0;
  const int* npart = nullptr;            // partial sums per matrix (= its W tiles)
  // host copies of the three prefix arrays (needed only to step a sub-range of the list)
  std::vector<int> h_proj_tile_start, h_row_start, h_w_tile_start;
};

// Enqueues the six phases for the matrices [qa, qb) of the list (qb < 0: the whole list); returns
// the number of launches.
int launch_simt_step(const SimtPlan& pl, const Hyper& hp, unsigned* status_dev, cudaStream_t st,
                     PhaseTimer* tm, int qa = 0, int qb = -1);
extern const char* const kSimtPhaseNames[6];

// One block of 256 threads per matrix of the list: sums the matrix's partial sums
// of ||S||^2 (npart_of[i] floats at mt.part) in a fixed order, applies the limiter
// rule (Eq. 12 in Algorithm 1's form), stores lambda and the new ||S_prev||,
// records the range of k and advances t.
__global__ void k_finalize(const MatDev* __restrict__ mats, const int* __restrict__ list, int nlist,
                           const int* __restrict__ npart_of, Hyper hp, unsigned* __restrict__ status);

// Fira-only-scaling, element-wise over tiles of `tile` x `tile` elements of W (one block of 256
// threads per tile; tile_start holds nlist + 1 ascending tile counts; `first` is added to the
// block index, `tiles` blocks are launched).  update = 0: part[tile] = sum over the tile of (k_l G)^2, the norm that the
// limiter sees; update = 1: W <- W - lr a_res lambda k_l G.
void launch_scaled_gradient(const MatDev* mats, const int* list, int nlist, const int* tile_start, int first,
                            int tiles, int tile, int update, float lr, float a_res, cudaStream_t st);

}  // namespace fira
