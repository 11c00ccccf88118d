// bf16 tensor-core step kernels (placeholder until the tcgen05 path lands: every
// matrix is routed to the fp32 CUDA-core kernels).
#include "context.cuh"
#include "step_tc.cuh"

namespace fira {

bool tc_supported(const fira_matrix_desc&) { return false; }
size_t tc_colpart_floats(const fira_matrix_desc&) { return 0; }
size_t tc_part_floats(const fira_matrix_desc&) { return 0; }
fira_status tc_build_plan(fira_ctx*, std::vector<int>&) { return FIRA_OK; }
void tc_destroy_plan(fira_ctx*) {}
fira_status tc_update_pointers(fira_ctx*) { return FIRA_OK; }
int launch_tc_step(fira_ctx*, const Hyper&) { return 0; }
int tc_phase_names(const char**) { return 0; }

}  // namespace fira
