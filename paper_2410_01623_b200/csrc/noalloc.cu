// fira_step_single_noalloc(): one Fira step of one matrix for callers that cannot
// allocate device memory.
//
// Who needs this.  Code that runs where cudaMalloc is off limits: a plug-in called
// from inside another framework's memory pool that forbids side allocations, a
// real-time loop that must not touch the driver's allocator, an environment whose
// memory budget was fixed at start-up.  Such a caller cannot supply the state and
// scratch buffers that fira_init() asks for, so the intermediates of the step live
// in a fixed array that is part of the library image instead.
//
// The array costs kNoAllocScratchBytes on every GPU that loads the library, for the
// life of the process.  All calls share it and it keeps what the previous call left
// there: two calls that overlap on the GPU (different streams, or different host
// threads) corrupt each other.  Each call rewrites whatever it reads from the array.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <mutex>

#include "context.cuh"
#include "simt_gemm.cuh"

namespace fira {

namespace {

constexpr size_t kNoAllocScratchBytes = 8u << 20;   // 8 MiB
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
// Device addresses of g_noalloc_scratch, one per device, resolved on first use.  In
// host code the name g_noalloc_scratch is only a handle for the runtime; the address
// a kernel may dereference comes from cudaGetSymbolAddress on the current device.
unsigned char* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_addr_mutex;   // several host threads may reach the look-up at once

// Device address of the array on the current device (looked up once per device, with
// that device current); null on error, with the message set.
unsigned char* scratch_base() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    set_error(std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_scratch_addr_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) {
      set_error(std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
      return nullptr;
    }
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  return g_scratch_addr[dev];
}

struct Carve {
  size_t off_mats, off_status, off_ints, off_sc, off_rt, off_xt, off_k, off_part, total;
};

Carve carve(int m, int n, int r) {
  const size_t l = std::max(m, n);
  const size_t tiles = (size_t)simt_tiles(m) * simt_tiles(n);
  Carve c;
  size_t o = 0;
  c.off_mats = o; o += align_up(sizeof(MatDev));
  c.off_status = o; o += 256;
  c.off_ints = o; o += 256;
  c.off_sc = o; o += align_up(sizeof(MatScalars));
  c.off_rt = o; o += align_up(l * r * 4);
  c.off_xt = o; o += align_up(l * r * 4);
  c.off_k = o; o += align_up(l * 4);
  c.off_part = o; o += align_up(tiles * 4);
  c.total = o;
  return c;
}

// The schedule arrays of a one-matrix list: [list(1)] [proj_start(2)] [row_start(2)] [w_start(2)] [npart(1)].
struct NoAllocInts { int v[8]; };

// Writes this call's tables into the array (it still holds the previous call's; everything else
// that a step reads there is rewritten by the step's own kernels before it is read).  The matrix
// record and the schedule arrays travel as kernel arguments, so that no host memory is referenced
// once the call has returned.  Also moves the two state scalars from the caller's memory into the
// MatScalars block that the step kernels use.
__global__ void k_noalloc_setup(MatDev mt, NoAllocInts ints, MatDev* mats_out, int* ints_out,
                                const float* norm_prev, const long long* t) {
  *mats_out = mt;
  for (int i = 0; i < 8; ++i) ints_out[i] = ints.v[i];
  MatScalars* sc = mt.sc;
  sc->prev_norm = (*norm_prev < 0.f) ? -1.f : *norm_prev;
  sc->lambda = 1.f; sc->norm_scaled = 0.f; sc->k_min = 0.f; sc->k_max = 0.f; sc->pad = 0.f;
  sc->t = *t;
}
__global__ void k_noalloc_store_scalars(const MatScalars* sc, float* norm_prev, long long* t) {
  *norm_prev = sc->prev_norm;
  *t = sc->t;
}

}  // namespace
}  // namespace fira

using namespace fira;

extern "C" fira_status fira_step_single_noalloc(const fira_hparams* hp, const fira_matrix_desc* desc,
                                                void* W_dev, const void* G_dev, const void* P_dev,
                                                float* M_dev, float* V_dev, float* norm_prev_dev,
                                                int64_t* t_dev, float lr, void* cuda_stream) {
  // every check comes before the first enqueue: a rejected call leaves the shared array as it was
  fira_status vs = validate(hp, desc, 1);
  if (vs != FIRA_OK) return vs;
  if (!W_dev || !G_dev || !P_dev || !M_dev || !V_dev || !norm_prev_dev || !t_dev) {
    set_error("null device pointer");
    return FIRA_ERR_INVALID_ARG;
  }
  if (((uintptr_t)W_dev | (uintptr_t)G_dev | (uintptr_t)P_dev | (uintptr_t)M_dev | (uintptr_t)V_dev) & 15) {
    set_error("W, G, P, M and V must be 16-byte aligned");
    return FIRA_ERR_INVALID_ARG;
  }
  if (!(lr < 0.f) && !isfinite(lr)) { set_error("lr must be finite"); return FIRA_ERR_INVALID_ARG; }
  if (hp->flags & (FIRA_FLAG_MATRIX_SCALING | FIRA_FLAG_NO_SCALING | FIRA_FLAG_NO_RESIDUAL | FIRA_FLAG_PSI_RMSPROP |
                   FIRA_FLAG_PSI_ADAGRAD | FIRA_FLAG_ONLY_SCALING)) {
    set_error("fira_step_single_noalloc: the variant flags are not supported by this entry point");
    return FIRA_ERR_UNSUPPORTED;
  }
  const Carve cv = carve(desc->m, desc->n, desc->r);
  if (cv.total > kNoAllocScratchBytes) {
    set_error("fira_step_single_noalloc: this matrix needs " + std::to_string(cv.total) +
              " bytes of scratch, the built-in array holds " + std::to_string(kNoAllocScratchBytes) +
              " (roughly max(m,n) * r <= 1,000,000)");
    return FIRA_ERR_WORKSPACE_TOO_SMALL;
  }
  unsigned char* base = scratch_base();
  if (!base) return FIRA_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  MatDev mt;
  memset(&mt, 0, sizeof(mt));
  mt.W = W_dev; mt.G = G_dev; mt.P = const_cast<void*>(P_dev); mt.M = M_dev; mt.V = V_dev;
  mt.sc = reinterpret_cast<MatScalars*>(base + cv.off_sc);
  mt.Rt = reinterpret_cast<float*>(base + cv.off_rt);
  mt.Xt = reinterpret_cast<float*>(base + cv.off_xt);
  mt.kvec = reinterpret_cast<float*>(base + cv.off_k);
  mt.part = reinterpret_cast<float*>(base + cv.off_part);
  mt.m = desc->m; mt.n = desc->n; mt.r = desc->r;
  mt.ld = desc->ld ? desc->ld : desc->n;
  mt.left = desc->m <= desc->n;
  mt.bf16 = desc->dtype == FIRA_BF16;
  mt.l = std::max(desc->m, desc->n); mt.d = std::min(desc->m, desc->n);
  mt.engine = 0;

  const int ptiles = simt_tiles(mt.l) * simt_tiles(mt.r);
  const int wtiles = simt_tiles(mt.m) * simt_tiles(mt.n);
  const NoAllocInts ints = {{0, 0, ptiles, 0, mt.l, 0, wtiles, wtiles}};
  int* ints_dev = reinterpret_cast<int*>(base + cv.off_ints);
  // sticky across calls until fira_noalloc_poll() reads it (zero when the library is loaded)
  unsigned* status_dev = reinterpret_cast<unsigned*>(base + cv.off_status);

  k_noalloc_setup<<<1, 1, 0, st>>>(mt, ints, reinterpret_cast<MatDev*>(base + cv.off_mats), ints_dev,
                                   norm_prev_dev, reinterpret_cast<const long long*>(t_dev));
  SimtPlan pl;
  pl.mats = reinterpret_cast<const MatDev*>(base + cv.off_mats);
  pl.list = ints_dev; pl.nlist = 1;
  pl.proj_tile_start = ints_dev + 1; pl.proj_tiles = ptiles;
  pl.row_start = ints_dev + 3; pl.rows_total = mt.l;
  pl.w_tile_start = ints_dev + 5; pl.w_tiles = wtiles;
  pl.npart = ints_dev + 7;
  Hyper h;
  h.beta1 = hp->beta1; h.beta2 = hp->beta2; h.eps = hp->eps;
  h.lr = lr < 0.f ? hp->lr : lr;
  h.a_low = hp->alpha;
  h.a_res = (hp->flags & FIRA_FLAG_ALPHA_LOWRANK_ONLY) ? 1.f : hp->alpha;
  h.mode = 0;
  h.gamma = hp->gamma;
  PhaseTimer no_timer;
  launch_simt_step(pl, h, status_dev, st, &no_timer);
  k_noalloc_store_scalars<<<1, 1, 0, st>>>(mt.sc, norm_prev_dev, reinterpret_cast<long long*>(t_dev));
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_error(std::string("fira_step_single_noalloc: ") + cudaGetErrorString(e));
    return FIRA_ERR_CUDA;
  }
  return FIRA_OK;
}

extern "C" size_t fira_noalloc_max_scratch_bytes(void) { return kNoAllocScratchBytes; }

extern "C" fira_status fira_noalloc_poll(void* cuda_stream) {
  unsigned char* base = scratch_base();
  if (!base) return FIRA_ERR_CUDA;
  // the status word sits at the same offset for every matrix size
  unsigned* status_dev = reinterpret_cast<unsigned*>(base + carve(1, 1, 1).off_status);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, status_dev, sizeof(v), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess && v != 0) e = cudaMemsetAsync(status_dev, 0, sizeof(unsigned), st);
  if (e != cudaSuccess) { set_error(std::string("fira_noalloc_poll: ") + cudaGetErrorString(e)); return FIRA_ERR_CUDA; }
  if (v & DEV_STATUS_NONFINITE) { set_error("a non-finite norm or factor was produced"); return FIRA_ERR_NONFINITE; }
  if (v & DEV_STATUS_TIMEOUT) { set_error("a bounded device-side wait ran out"); return FIRA_ERR_DEVICE_TIMEOUT; }
  return FIRA_OK;
}
