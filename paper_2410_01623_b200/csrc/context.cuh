// Host-side context of the Fira library (private to the library).
#pragma once
#include "common.cuh"
#include "step_simt.cuh"

namespace fira { struct TcPlan; }

namespace fira {
// Streams and events of fira_step_host(): created on its first call.
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, out_done = nullptr;
  std::vector<cudaEvent_t> in_done, stepped;     // per chunk
};
}  // namespace fira

struct fira_ctx {
  fira_hparams hp;
  std::vector<fira_matrix_desc> descs;
  std::vector<fira::MatDev> mats;        // host mirror of the device table
  cudaStream_t stream = nullptr;
  int device = 0;

  char* state_base = nullptr;
  size_t state_bytes = 0;
  char* scratch_base = nullptr;
  size_t scratch_bytes = 0;

  // sections inside the scratch buffer
  fira::MatDev* mats_dev = nullptr;
  unsigned* status_dev = nullptr;
  char* tc_maps_dev = nullptr;           // tensor maps of the tensor-core path
  int* ints_dev = nullptr;               // all schedule arrays, one block
  size_t ints_count = 0;
  char* work_base = nullptr;             // per-matrix step scratch, reused by the refresh
  size_t work_bytes = 0;

  fira::SimtPlan simt;                   // matrices on the fp32 CUDA-core kernels
  fira::TcPlan* tc = nullptr;            // matrices on the tensor-core kernels
  std::vector<int> simt_list, tc_list;
  std::vector<long long> t_host;         // host mirror of every matrix's step count
  fira::PhaseTimer timer;
  fira::HostPipe pipe;
  bool table_dirty = true;
  bool proj_weights_dirty = true;        // tensor-core path: column norms of the stored projections to be retaken
  int last_launches = 0;
};

namespace fira {

struct Layout {
  // byte offsets per matrix inside the state buffer
  std::vector<size_t> offP, offM, offV, offS;
  size_t state_bytes = 0;
  // byte offsets inside the scratch buffer
  size_t off_mats = 0, off_status = 0, off_ints = 0, off_tcmaps = 0, off_work = 0;
  size_t ints_count = 0;
  // byte offsets per matrix inside the work area
  std::vector<size_t> offRt, offXt, offK, offPart, offNb, offRb, offXb, offColpart, offGs, offWs, offAux;
  std::vector<int> engine;
  size_t step_work_bytes = 0, refresh_min_bytes = 0;
  size_t scratch_bytes = 0;
};

fira_status validate(const fira_hparams* hp, const fira_matrix_desc* descs, int32_t count);
Layout make_layout(const fira_hparams& hp, const fira_matrix_desc* descs, int32_t count);
size_t refresh_bytes_per_matrix(const fira_matrix_desc& d);
int engine_for(const fira_hparams& hp, const fira_matrix_desc& d);

// Where a refresh works and where its result goes.  Default: the context's own work area and
// stream, the bases stored into the context's projections.  The side variant: a work buffer and a
// stream of the caller's, the bases written to the caller's buffers (per matrix index, in the
// matrix's storage type) and nothing of the context modified, so that it may run next to steps.
struct RefreshTarget {
  char* work_base = nullptr;
  size_t work_bytes = 0;
  cudaStream_t stream = nullptr;
  void* const* P_out = nullptr;      // null: the context's projections
};
fira_status refresh_impl(fira_ctx* ctx, const void* const* G_dev, const std::vector<int>& which,
                         uint64_t seed, int iters, float* const* basis_out = nullptr,
                         const RefreshTarget* target = nullptr);

}  // namespace fira
