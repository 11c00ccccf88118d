// Launch interface of the bf16 tensor-core (tcgen05) step kernels.
#pragma once
#include <vector>

#include "common.cuh"

struct fira_ctx;

namespace fira {

// Whether the tensor-core kernels can take this matrix (type, rank and size rules of the
// tiles); otherwise it runs on the fp32 CUDA-core kernels.
bool tc_supported(const fira_matrix_desc& d);
// Row pitch (elements) of the aligned copies of G and W that the tensor-core path makes when the
// caller's rows are not 16-byte aligned (odd widths or pitches); 0 when TMA can read them in place.
long long tc_staging_pitch(const fira_matrix_desc& d, uint32_t flags);
bool tc_rows_aligned(const fira_matrix_desc& d);
// Scratch sizes (floats) of the per-(r-tile, l) column partial sums and of the
// partial sums of ||S||^2.
size_t tc_colpart_floats(const fira_matrix_desc& d);
size_t tc_part_floats(const fira_matrix_desc& d);
// Bytes of this engine's device-resident tables (tensor maps, tile records) for a matrix list.
size_t tc_tables_bytes(const fira_hparams& hp, const fira_matrix_desc* descs, int count);
// Appends this engine's schedule arrays to `ints` (host image of the device int
// block) and records where they are.
fira_status tc_build_plan(fira_ctx* c, std::vector<int>& ints);
void tc_destroy_plan(fira_ctx* c);
// Called when W / G pointers changed: re-encodes what depends on them.
fira_status tc_update_pointers(fira_ctx* c);
// Enqueues the tensor-core phases for the matrices [qa, qb) of the tc list (qb < 0: all of it);
// returns the number of launches (negative: error, message set).
int launch_tc_step(fira_ctx* c, const Hyper& hp, int qa = 0, int qb = -1);
// Launches the self-test kernel of the bounded waits (one block; sets the time-out bit of the
// context's status word after `rounds` tries on a barrier that nothing arrives on).
fira_status tc_selftest_bounded_wait(fira_ctx* c, int rounds);
// Names of this engine's phases in launch order (8).
int tc_phase_names(const char** out);

// ---- products of the projection refresh on the tensor cores
// C[l][j] (fp32, L x r) = sum over k < D of A(k, l) B[k][j], with A taken in place from the bf16
// matrix G (m x n, pitch ld, rows 16-byte aligned): mn_major = 1: G is [k][l] (D = m, L = n);
// mn_major = 0: G is [l][k] (L = m, D = n).  B is bf16 [D][r].  r % 128 == 0.
// Split-precision products: with nseg > 1 the product runs over nseg k-segments that accumulate into
// the same output; segment s takes A from G (bit s of asel clear) or G_lo (set) and B from B (bsel
// clear) or B_lo (set).  G_lo / B_lo have the shapes and pitches of G / B.  For an fp32 matrix
// X = X_hi + X_lo (two bf16 parts), segments (hi,hi), (hi,lo), (lo,hi) give X Y to about 2^-16.
struct TcGemmJob {
  const void* G; long long ld; int m, n; int mn_major;
  const void* B; float* C; int r;
  const void* G_lo; const void* B_lo;
  int nseg; unsigned asel, bsel;
};
// Device bytes of the tables (tensor maps, tile records) of a job list.
size_t tc_gemm_table_bytes(const TcGemmJob* jobs, int njobs);
// Builds the tables on the host and uploads them to table_dev (256-byte aligned) on the given
// stream; *ntiles_out is what tc_gemm_run needs.
fira_status tc_gemm_prepare(fira_ctx* c, const TcGemmJob* jobs, int njobs, char* table_dev, size_t table_bytes,
                            int* ntiles_out, cudaStream_t st);
// One grouped launch over the prepared jobs.
fira_status tc_gemm_run(fira_ctx* c, const char* table_dev, int njobs, int ntiles, cudaStream_t st);

}  // namespace fira
