// C-ABI entry points of the Fira library: argument checks, buffer carving, the
// device problem table and the per-step launch sequence.  All arithmetic of the
// method runs in the kernels of step_simt.cu, step_tc.cu and refresh.cu.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "context.cuh"
#include "simt_gemm.cuh"
#include "step_tc.cuh"

namespace fira {

static thread_local std::string g_last_error;
void set_error(const std::string& msg) { g_last_error = msg; }

#define FIRA_CUDA(call)                                                        \
  do {                                                                         \
    cudaError_t e_ = (call);                                                   \
    if (e_ != cudaSuccess) {                                                   \
      set_error(std::string(#call) + ": " + cudaGetErrorString(e_));           \
      return FIRA_ERR_CUDA;                                                    \
    }                                                                          \
  } while (0)

fira_status validate(const fira_hparams* hp, const fira_matrix_desc* descs, int32_t count) {
  if (!hp || !descs || count <= 0) { set_error("null argument or empty matrix list"); return FIRA_ERR_INVALID_ARG; }
  if (!(hp->eps > 0.f) || !isfinite(hp->eps)) { set_error("eps must be > 0"); return FIRA_ERR_INVALID_ARG; }
  if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f)) {
    set_error("beta1, beta2 must lie in [0, 1)"); return FIRA_ERR_INVALID_ARG;
  }
  if (isnan(hp->gamma) || hp->gamma < 1.f) { set_error("gamma must be >= 1 or +inf"); return FIRA_ERR_INVALID_ARG; }
  if (!isfinite(hp->lr) || !isfinite(hp->alpha)) { set_error("lr and alpha must be finite"); return FIRA_ERR_INVALID_ARG; }
  if (hp->T < 0) { set_error("T must be >= 0"); return FIRA_ERR_INVALID_ARG; }
  if ((hp->flags & FIRA_FLAG_MATRIX_SCALING) && (hp->flags & FIRA_FLAG_NO_SCALING)) {
    set_error("FIRA_FLAG_MATRIX_SCALING and FIRA_FLAG_NO_SCALING exclude each other"); return FIRA_ERR_INVALID_ARG;
  }
  if ((hp->flags & FIRA_FLAG_PSI_RMSPROP) && (hp->flags & FIRA_FLAG_PSI_ADAGRAD)) {
    set_error("FIRA_FLAG_PSI_RMSPROP and FIRA_FLAG_PSI_ADAGRAD exclude each other"); return FIRA_ERR_INVALID_ARG;
  }
  if ((hp->flags & FIRA_FLAG_ONLY_SCALING) && (hp->flags & FIRA_FLAG_NO_RESIDUAL)) {
    set_error("FIRA_FLAG_ONLY_SCALING and FIRA_FLAG_NO_RESIDUAL exclude each other"); return FIRA_ERR_INVALID_ARG;
  }
  for (int i = 0; i < count; ++i) {
    const fira_matrix_desc& d = descs[i];
    if (d.m <= 0 || d.n <= 0 || d.r <= 0 || d.r > std::min(d.m, d.n)) {
      set_error("matrix " + std::to_string(i) + ": need m, n > 0 and 1 <= r <= min(m, n)");
      return FIRA_ERR_INVALID_ARG;
    }
    if (d.dtype != FIRA_F32 && d.dtype != FIRA_BF16) { set_error("unknown dtype"); return FIRA_ERR_INVALID_ARG; }
    if (d.ld != 0 && d.ld < d.n) { set_error("ld must be 0 or >= n"); return FIRA_ERR_INVALID_ARG; }
  }
  return FIRA_OK;
}

int engine_for(const fira_hparams& hp, const fira_matrix_desc& d) {
  if (d.dtype != FIRA_BF16 || (hp.flags & FIRA_FLAG_FORCE_SIMT)) return 0;
  return tc_supported(d) ? 1 : 0;
}

Layout make_layout(const fira_hparams& hp, const fira_matrix_desc* descs, int32_t count) {
  Layout L;
  size_t so = 0;
  L.engine.resize(count);
  for (int i = 0; i < count; ++i) {
    const fira_matrix_desc& d = descs[i];
    const size_t dd = std::min(d.m, d.n), ll = std::max(d.m, d.n), r = d.r;
    const size_t es = d.dtype == FIRA_BF16 ? 2 : 4;
    L.offP.push_back(so); so += align_up(dd * r * es);
    L.offM.push_back(so); so += align_up(ll * r * 4);
    L.offV.push_back(so); so += align_up(ll * r * 4);
    L.offS.push_back(so); so += align_up(sizeof(MatScalars));
    L.engine[i] = engine_for(hp, d);
  }
  L.state_bytes = so;
  size_t wo = 0;
  L.off_mats = wo; wo += align_up(sizeof(MatDev) * count);
  L.off_status = wo; wo += 256;
  L.ints_count = 16 * (size_t)(count + 1);
  L.off_ints = wo; wo += align_up(L.ints_count * sizeof(int));
  L.off_tcmaps = wo; wo += tc_tables_bytes(hp, descs, count);
  L.off_work = wo;
  size_t w = 0;
  size_t refresh_max = 0;
  L.offRt.assign(count, 0); L.offXt.assign(count, 0); L.offK.assign(count, 0); L.offPart.assign(count, 0);
  L.offNb.assign(count, 0); L.offRb.assign(count, 0); L.offXb.assign(count, 0);
  L.offColpart.assign(count, 0); L.offGs.assign(count, 0); L.offWs.assign(count, 0); L.offAux.assign(count, 0);
  for (int i = 0; i < count; ++i) {
    fira_matrix_desc d = descs[i];
    if (d.ld == 0) d.ld = d.n;
    const size_t ll = std::max(d.m, d.n), r = d.r;
    L.offK[i] = w; w += align_up(ll * 4);
    L.offAux[i] = w; w += align_up(2 * ll * 4);
    if (L.engine[i] == 0) {
      const size_t tiles = (size_t)simt_tiles(d.m) * simt_tiles(d.n);
      L.offRt[i] = w; w += align_up(ll * r * 4);
      L.offXt[i] = w; w += align_up(ll * r * 4);
      L.offPart[i] = w; w += align_up(tiles * 4);
    } else {
      L.offNb[i] = w; w += align_up(ll * r * 2);
      L.offRb[i] = w; w += align_up(ll * r * 2);
      L.offXb[i] = w; w += align_up(ll * r * 2);
      L.offColpart[i] = w; w += align_up(tc_colpart_floats(d) * 4);
      L.offPart[i] = w; w += align_up(tc_part_floats(d) * 4);
      const size_t lds = (size_t)tc_staging_pitch(d, hp.flags);
      if (lds) {
        L.offGs[i] = w; w += align_up((size_t)d.m * lds * 2);
        L.offWs[i] = w; w += align_up((size_t)d.m * lds * 2);
      }
    }
    refresh_max = std::max(refresh_max, refresh_bytes_per_matrix(d));
  }
  L.step_work_bytes = w;
  L.refresh_min_bytes = refresh_max;
  L.scratch_bytes = L.off_work + std::max(L.step_work_bytes, L.refresh_min_bytes);
  return L;
}

static fira_status upload_table(fira_ctx* c) {
  FIRA_CUDA(cudaMemcpyAsync(c->mats_dev, c->mats.data(), sizeof(MatDev) * c->mats.size(),
                            cudaMemcpyHostToDevice, c->stream));
  c->table_dirty = false;
  return FIRA_OK;
}

static Hyper make_hyper(const fira_hparams& hp, float lr) {
  Hyper h;
  h.beta1 = hp.beta1; h.beta2 = hp.beta2; h.eps = hp.eps;
  h.lr = lr < 0.f ? hp.lr : lr;
  h.a_low = hp.alpha;
  h.a_res = (hp.flags & FIRA_FLAG_ALPHA_LOWRANK_ONLY) ? 1.f : hp.alpha;
  h.mode = 0;
  if (hp.flags & FIRA_FLAG_MATRIX_SCALING) h.mode |= HYPER_MATRIX_SCALING;
  if (hp.flags & FIRA_FLAG_NO_SCALING) h.mode |= HYPER_NO_SCALING;
  if (hp.flags & FIRA_FLAG_NO_RESIDUAL) { h.mode |= HYPER_NO_RESIDUAL; h.a_res = 0.f; }
  if (hp.flags & FIRA_FLAG_PSI_RMSPROP) h.mode |= HYPER_PSI_RMSPROP;
  if (hp.flags & FIRA_FLAG_PSI_ADAGRAD) h.mode |= HYPER_PSI_ADAGRAD;
  if (hp.flags & FIRA_FLAG_ONLY_SCALING) h.mode |= HYPER_ONLY_SCALING;
  h.gamma = hp.gamma;
  return h;
}

static size_t matrix_bytes(const MatDev& mt) { return (size_t)mt.m * mt.ld * (mt.bf16 ? 2 : 4); }

}  // namespace fira

using namespace fira;

extern "C" {

fira_status fira_query_workspace(const fira_hparams* hp, const fira_matrix_desc* descs, int32_t count,
                                 size_t* state_bytes, size_t* scratch_bytes) {
  fira_status s = validate(hp, descs, count);
  if (s != FIRA_OK) return s;
  if (!state_bytes || !scratch_bytes) { set_error("null output pointer"); return FIRA_ERR_INVALID_ARG; }
  Layout L = make_layout(*hp, descs, count);
  *state_bytes = L.state_bytes;
  *scratch_bytes = L.scratch_bytes;
  return FIRA_OK;
}

fira_status fira_init(fira_ctx** out, const fira_hparams* hp, const fira_matrix_desc* descs, int32_t count,
                      void* state_dev, size_t state_bytes, void* scratch_dev, size_t scratch_bytes,
                      void* cuda_stream) {
  if (!out) { set_error("null output pointer"); return FIRA_ERR_INVALID_ARG; }
  *out = nullptr;
  fira_status s = validate(hp, descs, count);
  if (s != FIRA_OK) return s;
  if (!state_dev || !scratch_dev || ((uintptr_t)state_dev & 255) || ((uintptr_t)scratch_dev & 255)) {
    set_error("state and scratch buffers must be non-null and 256-byte aligned");
    return FIRA_ERR_INVALID_ARG;
  }
  Layout L = make_layout(*hp, descs, count);
  if (state_bytes < L.state_bytes || scratch_bytes < L.scratch_bytes) {
    set_error("workspace too small: need state " + std::to_string(L.state_bytes) + " B, scratch " +
              std::to_string(L.scratch_bytes) + " B");
    return FIRA_ERR_WORKSPACE_TOO_SMALL;
  }
  fira_ctx* c = new (std::nothrow) fira_ctx();
  if (!c) { set_error("out of host memory"); return FIRA_ERR_INVALID_ARG; }
  c->hp = *hp;
  c->descs.assign(descs, descs + count);
  c->stream = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaGetDevice(&c->device);
  if (e != cudaSuccess) { set_error(std::string("cudaGetDevice: ") + cudaGetErrorString(e)); delete c; return FIRA_ERR_CUDA; }
  c->state_base = (char*)state_dev; c->state_bytes = state_bytes;
  c->scratch_base = (char*)scratch_dev; c->scratch_bytes = scratch_bytes;
  c->mats_dev = (MatDev*)(c->scratch_base + L.off_mats);
  c->status_dev = (unsigned*)(c->scratch_base + L.off_status);
  c->ints_dev = (int*)(c->scratch_base + L.off_ints);
  c->ints_count = L.ints_count;
  c->tc_maps_dev = c->scratch_base + L.off_tcmaps;
  c->work_base = c->scratch_base + L.off_work;
  c->work_bytes = scratch_bytes - L.off_work;

  c->mats.resize(count);
  c->t_host.assign(count, 0);
  for (int i = 0; i < count; ++i) {
    const fira_matrix_desc& d = descs[i];
    MatDev& mt = c->mats[i];
    memset(&mt, 0, sizeof(mt));
    mt.m = d.m; mt.n = d.n; mt.r = d.r;
    mt.ld = d.ld ? d.ld : d.n;
    c->descs[i].ld = mt.ld;
    mt.left = d.m <= d.n;
    mt.bf16 = d.dtype == FIRA_BF16;
    mt.l = std::max(d.m, d.n); mt.d = std::min(d.m, d.n);
    mt.engine = L.engine[i];
    mt.P = c->state_base + L.offP[i];
    mt.M = (float*)(c->state_base + L.offM[i]);
    mt.V = (float*)(c->state_base + L.offV[i]);
    mt.sc = (MatScalars*)(c->state_base + L.offS[i]);
    mt.kvec = (float*)(c->work_base + L.offK[i]);
    mt.aux = (float*)(c->work_base + L.offAux[i]);
    mt.part = (float*)(c->work_base + L.offPart[i]);
    if (mt.engine == 0) {
      mt.Rt = (float*)(c->work_base + L.offRt[i]);
      mt.Xt = (float*)(c->work_base + L.offXt[i]);
      c->simt_list.push_back(i);
    } else {
      mt.Nb = (__nv_bfloat16*)(c->work_base + L.offNb[i]);
      mt.Rb = (__nv_bfloat16*)(c->work_base + L.offRb[i]);
      mt.Xb = (__nv_bfloat16*)(c->work_base + L.offXb[i]);
      mt.colpart = (float*)(c->work_base + L.offColpart[i]);
      mt.lds = tc_staging_pitch(c->descs[i], c->hp.flags);
      if (mt.lds) {
        mt.Gs = (__nv_bfloat16*)(c->work_base + L.offGs[i]);
        mt.Ws = (__nv_bfloat16*)(c->work_base + L.offWs[i]);
      }
      c->tc_list.push_back(i);
    }
  }

  // schedule arrays: prefix sums over each engine's list
  std::vector<int> ints;
  auto push_block = [&](const std::vector<int>& v) {
    size_t o = ints.size();
    ints.insert(ints.end(), v.begin(), v.end());
    return o;
  };
  {
    const std::vector<int>& lst = c->simt_list;
    std::vector<int> pt{0}, rs{0}, wt{0}, np;
    for (int i : lst) {
      const MatDev& mt = c->mats[i];
      pt.push_back(pt.back() + simt_tiles(mt.l) * simt_tiles(mt.r));
      rs.push_back(rs.back() + mt.l);
      const int tiles = simt_tiles(mt.m) * simt_tiles(mt.n);
      wt.push_back(wt.back() + tiles);
      np.push_back(tiles);
    }
    const size_t o_list = push_block(lst), o_pt = push_block(pt), o_rs = push_block(rs),
                 o_wt = push_block(wt), o_np = push_block(np);
    c->simt.mats = c->mats_dev;
    c->simt.list = c->ints_dev + o_list; c->simt.nlist = (int)lst.size();
    c->simt.proj_tile_start = c->ints_dev + o_pt; c->simt.proj_tiles = pt.back();
    c->simt.row_start = c->ints_dev + o_rs; c->simt.rows_total = rs.back();
    c->simt.w_tile_start = c->ints_dev + o_wt; c->simt.w_tiles = wt.back();
    c->simt.npart = c->ints_dev + o_np;
    c->simt.h_proj_tile_start = pt; c->simt.h_row_start = rs; c->simt.h_w_tile_start = wt;
  }
  fira_status ts = tc_build_plan(c, ints);
  if (ts != FIRA_OK) { tc_destroy_plan(c); delete c; return ts; }
  if (ints.size() > c->ints_count) { set_error("internal: schedule arrays overflow"); tc_destroy_plan(c); delete c; return FIRA_ERR_INVALID_ARG; }

  cudaError_t ce = cudaSuccess;
  if (!ints.empty()) ce = cudaMemcpyAsync(c->ints_dev, ints.data(), ints.size() * sizeof(int), cudaMemcpyHostToDevice, c->stream);
  if (ce == cudaSuccess) ce = cudaMemsetAsync(c->state_base, 0, L.state_bytes, c->stream);
  if (ce == cudaSuccess) ce = cudaMemsetAsync(c->status_dev, 0, 256, c->stream);
  // ||S_prev|| = -1 marks "unset"
  MatScalars init;
  memset(&init, 0, sizeof(init));
  init.prev_norm = -1.f; init.lambda = 1.f;
  for (int i = 0; i < count && ce == cudaSuccess; ++i)
    ce = cudaMemcpyAsync(c->mats[i].sc, &init, sizeof(MatScalars), cudaMemcpyHostToDevice, c->stream);
  if (ce == cudaSuccess) ce = cudaMemcpyAsync(c->mats_dev, c->mats.data(), sizeof(MatDev) * count, cudaMemcpyHostToDevice, c->stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(c->stream);   // host staging buffers die on return
  if (ce != cudaSuccess) { set_error(std::string("fira_init: ") + cudaGetErrorString(ce)); tc_destroy_plan(c); delete c; return FIRA_ERR_CUDA; }
  c->table_dirty = true;
  *out = c;
  return FIRA_OK;
}

// Registers the caller's W and G pointers (re-encoding what depends on them).
static fira_status set_pointers(fira_ctx* c, void* const* W_dev, const void* const* G_dev) {
  const int count = (int)c->mats.size();
  bool ptr_changed = false;
  for (int i = 0; i < count; ++i) {
    if (c->mats[i].W != W_dev[i] || c->mats[i].G != G_dev[i]) {
      c->mats[i].W = W_dev[i]; c->mats[i].G = G_dev[i];
      ptr_changed = true;
    }
  }
  if (ptr_changed) {
    c->table_dirty = true;
    fira_status s = tc_update_pointers(c);
    if (s != FIRA_OK) return s;
  }
  if (c->table_dirty) { fira_status s = upload_table(c); if (s != FIRA_OK) return s; }
  return FIRA_OK;
}

// Enqueues the step of the matrices [i0, i1) (both engines' lists are ascending, so the range maps
// to one sub-range of each); returns the number of launches or -1.
static int launch_range(fira_ctx* c, const Hyper& h, int i0, int i1, bool whole) {
  if (whole) {
    int launches = launch_simt_step(c->simt, h, c->status_dev, c->stream, &c->timer);
    if (c->simt.nlist == 0) c->timer.mark(c->stream);
    const int tcl = launch_tc_step(c, h);
    return tcl < 0 ? -1 : launches + tcl;
  }
  auto sub = [&](const std::vector<int>& lst, int& qa, int& qb) {
    qa = (int)(std::lower_bound(lst.begin(), lst.end(), i0) - lst.begin());
    qb = (int)(std::lower_bound(lst.begin(), lst.end(), i1) - lst.begin());
  };
  int qa, qb, launches = 0;
  sub(c->simt_list, qa, qb);
  if (qb > qa) launches += launch_simt_step(c->simt, h, c->status_dev, c->stream, &c->timer, qa, qb);
  sub(c->tc_list, qa, qb);
  if (qb > qa) {
    const int tcl = launch_tc_step(c, h, qa, qb);
    if (tcl < 0) return -1;
    launches += tcl;
  }
  return launches;
}

static fira_status check_step_args(fira_ctx* c, void* const* W, const void* const* G, float lr) {
  if (!c || !W || !G) { set_error("null argument"); return FIRA_ERR_INVALID_ARG; }
  if (!(lr < 0.f) && !isfinite(lr)) { set_error("lr must be finite"); return FIRA_ERR_INVALID_ARG; }
  return FIRA_OK;
}

fira_status fira_step(fira_ctx* c, void* const* W_dev, const void* const* G_dev, float lr) {
  fira_status as = check_step_args(c, W_dev, G_dev, lr);
  if (as != FIRA_OK) return as;
  const int count = (int)c->mats.size();
  for (int i = 0; i < count; ++i) {
    if (!W_dev[i] || !G_dev[i] || ((uintptr_t)W_dev[i] & 15) || ((uintptr_t)G_dev[i] & 15)) {
      set_error("matrix " + std::to_string(i) + ": W and G must be non-null and 16-byte aligned");
      return FIRA_ERR_INVALID_ARG;
    }
  }
  if ((c->hp.flags & FIRA_FLAG_AUTO_REFRESH) && c->hp.T > 0) {
    std::vector<int> due;
    for (int i = 0; i < count; ++i) if (c->t_host[i] % c->hp.T == 0) due.push_back(i);
    if (!due.empty()) {
      fira_status rs = refresh_impl(c, G_dev, due, 0x5eedULL + (uint64_t)c->t_host[due[0]], -1);
      if (rs != FIRA_OK) return rs;
    }
  }
  fira_status ps = set_pointers(c, W_dev, G_dev);
  if (ps != FIRA_OK) return ps;
  const Hyper h = make_hyper(c->hp, lr);
  c->timer.begin_step();
  const int launches = launch_range(c, h, 0, count, true);
  if (launches < 0) return FIRA_ERR_CUDA;
  if (c->timer.on) c->timer.steps += 1;
  c->last_launches = launches;
  for (int i = 0; i < count; ++i) c->t_host[i] += 1;
  FIRA_CUDA(cudaGetLastError());
  return FIRA_OK;
}

size_t fira_staging_bytes(const fira_ctx* c) {
  if (!c) return 0;
  size_t tot = 0;
  for (const MatDev& mt : c->mats) tot += 2 * align_up(matrix_bytes(mt));
  return tot;
}

fira_status fira_step_host(fira_ctx* c, void* const* W_host, const void* const* G_host, float lr,
                           void* staging_dev, size_t staging_bytes) {
  fira_status as = check_step_args(c, W_host, G_host, lr);
  if (as != FIRA_OK) return as;
  if (!staging_dev) { set_error("null argument"); return FIRA_ERR_INVALID_ARG; }
  if (((uintptr_t)staging_dev & 255) || staging_bytes < fira_staging_bytes(c)) {
    set_error("staging buffer must be 256-byte aligned and hold fira_staging_bytes() bytes");
    return FIRA_ERR_WORKSPACE_TOO_SMALL;
  }
  const int count = (int)c->mats.size();
  for (int i = 0; i < count; ++i)
    if (!W_host[i] || !G_host[i]) { set_error("null host matrix"); return FIRA_ERR_INVALID_ARG; }
  std::vector<void*> Wd(count);
  std::vector<const void*> Gd(count);
  size_t total = 0;
  {
    char* p = (char*)staging_dev;
    for (int i = 0; i < count; ++i) {
      const size_t bytes = matrix_bytes(c->mats[i]);
      Gd[i] = p; p += align_up(bytes);
      Wd[i] = p; p += align_up(bytes);
      total += bytes;
    }
  }
  // Chunks of consecutive matrices: while chunk q steps, chunk q + 1 is on its way in and the
  // weights of chunk q - 1 on their way out (the link carries both directions at once).  Two
  // side streams carry the copies; events order them against the context's stream.
  HostPipe& hp_ = c->pipe;
  if (!hp_.in) {
    FIRA_CUDA(cudaStreamCreateWithFlags(&hp_.in, cudaStreamNonBlocking));
    FIRA_CUDA(cudaStreamCreateWithFlags(&hp_.out, cudaStreamNonBlocking));
    FIRA_CUDA(cudaEventCreateWithFlags(&hp_.start, cudaEventDisableTiming));
    FIRA_CUDA(cudaEventCreateWithFlags(&hp_.out_done, cudaEventDisableTiming));
  }
  std::vector<int> cut{0};
  {
    const size_t target = std::max<size_t>(total / 32, (size_t)32 << 20);   // about 32 chunks, 32 MiB at least
    size_t acc = 0;
    for (int i = 0; i < count; ++i) {
      acc += matrix_bytes(c->mats[i]);
      if (acc >= target || i + 1 == count) { cut.push_back(i + 1); acc = 0; }
    }
  }
  const int nchunk = (int)cut.size() - 1;
  while ((int)hp_.in_done.size() < nchunk) {
    cudaEvent_t a, b;
    FIRA_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
    FIRA_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
    hp_.in_done.push_back(a); hp_.stepped.push_back(b);
  }
  if ((c->hp.flags & FIRA_FLAG_AUTO_REFRESH) && c->hp.T > 0) {
    set_error("fira_step_host: FIRA_FLAG_AUTO_REFRESH is not supported with host buffers (refresh needs G on the device)");
    return FIRA_ERR_UNSUPPORTED;
  }
  fira_status ps = set_pointers(c, Wd.data(), Gd.data());
  if (ps != FIRA_OK) return ps;
  const Hyper h = make_hyper(c->hp, lr);
  // the copies start once everything enqueued so far on the context's stream has run (an earlier
  // call's kernels may still be reading the staging buffer)
  FIRA_CUDA(cudaEventRecord(hp_.start, c->stream));
  FIRA_CUDA(cudaStreamWaitEvent(hp_.in, hp_.start, 0));
  FIRA_CUDA(cudaStreamWaitEvent(hp_.out, hp_.start, 0));
  c->timer.begin_step();
  int launches = 0;
  for (int q = 0; q < nchunk; ++q) {
    for (int i = cut[q]; i < cut[q + 1]; ++i) {
      const size_t bytes = matrix_bytes(c->mats[i]);
      FIRA_CUDA(cudaMemcpyAsync(const_cast<void*>(Gd[i]), G_host[i], bytes, cudaMemcpyHostToDevice, hp_.in));
      FIRA_CUDA(cudaMemcpyAsync(Wd[i], W_host[i], bytes, cudaMemcpyHostToDevice, hp_.in));
    }
    FIRA_CUDA(cudaEventRecord(hp_.in_done[q], hp_.in));
    FIRA_CUDA(cudaStreamWaitEvent(c->stream, hp_.in_done[q], 0));
    const int l = launch_range(c, h, cut[q], cut[q + 1], nchunk == 1);
    if (l < 0) return FIRA_ERR_CUDA;
    launches += l;
    FIRA_CUDA(cudaEventRecord(hp_.stepped[q], c->stream));
    FIRA_CUDA(cudaStreamWaitEvent(hp_.out, hp_.stepped[q], 0));
    for (int i = cut[q]; i < cut[q + 1]; ++i)
      FIRA_CUDA(cudaMemcpyAsync(W_host[i], Wd[i], matrix_bytes(c->mats[i]), cudaMemcpyDeviceToHost, hp_.out));
  }
  // the context's stream is done when the last weights have arrived
  FIRA_CUDA(cudaEventRecord(hp_.out_done, hp_.out));
  FIRA_CUDA(cudaStreamWaitEvent(c->stream, hp_.out_done, 0));
  c->last_launches = launches;
  for (int i = 0; i < count; ++i) c->t_host[i] += 1;
  FIRA_CUDA(cudaGetLastError());
  return FIRA_OK;
}

fira_status fira_refresh_projection(fira_ctx* c, const void* const* G_dev, const int32_t* which, int32_t nwhich,
                                    uint64_t seed, int32_t iters) {
  return fira_refresh_projection_f32(c, G_dev, which, nwhich, seed, iters, nullptr);
}

fira_status fira_refresh_projection_f32(fira_ctx* c, const void* const* G_dev, const int32_t* which, int32_t nwhich,
                                        uint64_t seed, int32_t iters, float* const* basis_f32_dev) {
  if (!c || !G_dev) { set_error("null argument"); return FIRA_ERR_INVALID_ARG; }
  const int count = (int)c->mats.size();
  std::vector<int> sel;
  if (!which) { for (int i = 0; i < count; ++i) sel.push_back(i); }
  else {
    if (nwhich < 0) { set_error("nwhich < 0"); return FIRA_ERR_INVALID_ARG; }
    for (int q = 0; q < nwhich; ++q) {
      if (which[q] < 0 || which[q] >= count) { set_error("matrix index out of range"); return FIRA_ERR_INVALID_ARG; }
      sel.push_back(which[q]);
    }
  }
  for (int i : sel) {
    if (!G_dev[i] || ((uintptr_t)G_dev[i] & 15)) { set_error("G must be non-null and 16-byte aligned"); return FIRA_ERR_INVALID_ARG; }
  }
  if (sel.empty()) return FIRA_OK;
  if (basis_f32_dev)
    for (int i : sel)
      if (basis_f32_dev[i] && ((uintptr_t)basis_f32_dev[i] & 15)) { set_error("basis output must be 16-byte aligned"); return FIRA_ERR_INVALID_ARG; }
  return refresh_impl(c, G_dev, sel, seed, iters, basis_f32_dev);
}

size_t fira_refresh_side_work_bytes(const fira_ctx* c) {
  if (!c) return 0;
  size_t mx = 0;
  for (const fira_matrix_desc& d : c->descs) mx = std::max(mx, refresh_bytes_per_matrix(d));
  return align_up(mx);
}

fira_status fira_refresh_projection_side(fira_ctx* c, const void* const* G_dev, const int32_t* which, int32_t nwhich,
                                         uint64_t seed, int32_t iters, void* const* P_out_dev, void* work_dev,
                                         size_t work_bytes, void* side_stream) {
  if (!c || !G_dev || !P_out_dev || !work_dev) { set_error("null argument"); return FIRA_ERR_INVALID_ARG; }
  const int count = (int)c->mats.size();
  std::vector<int> sel;
  if (!which) { for (int i = 0; i < count; ++i) sel.push_back(i); }
  else {
    if (nwhich < 0) { set_error("nwhich < 0"); return FIRA_ERR_INVALID_ARG; }
    for (int q = 0; q < nwhich; ++q) {
      if (which[q] < 0 || which[q] >= count) { set_error("matrix index out of range"); return FIRA_ERR_INVALID_ARG; }
      sel.push_back(which[q]);
    }
  }
  for (int i : sel) {
    if (!G_dev[i] || ((uintptr_t)G_dev[i] & 15)) { set_error("G must be non-null and 16-byte aligned"); return FIRA_ERR_INVALID_ARG; }
    if (!P_out_dev[i] || ((uintptr_t)P_out_dev[i] & 15)) { set_error("projection output must be non-null and 16-byte aligned"); return FIRA_ERR_INVALID_ARG; }
  }
  if (((uintptr_t)work_dev & 255) || work_bytes < fira_refresh_side_work_bytes(c)) {
    set_error("work buffer must be 256-byte aligned and hold fira_refresh_side_work_bytes() bytes");
    return FIRA_ERR_WORKSPACE_TOO_SMALL;
  }
  if (sel.empty()) return FIRA_OK;
  RefreshTarget tg;
  tg.work_base = (char*)work_dev; tg.work_bytes = work_bytes; tg.stream = (cudaStream_t)side_stream; tg.P_out = P_out_dev;
  return refresh_impl(c, G_dev, sel, seed, iters, nullptr, &tg);
}

static fira_status check_idx(const fira_ctx* c, int32_t idx) {
  if (!c) { set_error("null context"); return FIRA_ERR_INVALID_ARG; }
  if (idx < 0 || idx >= (int)c->mats.size()) { set_error("matrix index out of range"); return FIRA_ERR_INVALID_ARG; }
  return FIRA_OK;
}

fira_status fira_set_projection(fira_ctx* c, int32_t idx, const void* P_dev) {
  fira_status s = check_idx(c, idx); if (s != FIRA_OK) return s;
  if (!P_dev) { set_error("null projection"); return FIRA_ERR_INVALID_ARG; }
  const MatDev& mt = c->mats[idx];
  const size_t bytes = (size_t)mt.d * mt.r * (mt.bf16 ? 2 : 4);
  FIRA_CUDA(cudaMemcpyAsync(mt.P, P_dev, bytes, cudaMemcpyDeviceToDevice, c->stream));
  c->proj_weights_dirty = true;
  return FIRA_OK;
}

fira_status fira_get_projection(fira_ctx* c, int32_t idx, void* P_dev) {
  fira_status s = check_idx(c, idx); if (s != FIRA_OK) return s;
  if (!P_dev) { set_error("null projection"); return FIRA_ERR_INVALID_ARG; }
  const MatDev& mt = c->mats[idx];
  const size_t bytes = (size_t)mt.d * mt.r * (mt.bf16 ? 2 : 4);
  FIRA_CUDA(cudaMemcpyAsync(P_dev, mt.P, bytes, cudaMemcpyDeviceToDevice, c->stream));
  return FIRA_OK;
}

fira_status fira_get_state(fira_ctx* c, int32_t idx, float* M_dev, float* V_dev, float* norm_prev_host,
                           int64_t* t_host) {
  fira_status s = check_idx(c, idx); if (s != FIRA_OK) return s;
  const MatDev& mt = c->mats[idx];
  const size_t bytes = (size_t)mt.l * mt.r * 4;
  if (M_dev) FIRA_CUDA(cudaMemcpyAsync(M_dev, mt.M, bytes, cudaMemcpyDeviceToDevice, c->stream));
  if (V_dev) FIRA_CUDA(cudaMemcpyAsync(V_dev, mt.V, bytes, cudaMemcpyDeviceToDevice, c->stream));
  MatScalars sc;
  FIRA_CUDA(cudaMemcpyAsync(&sc, mt.sc, sizeof(sc), cudaMemcpyDeviceToHost, c->stream));
  FIRA_CUDA(cudaStreamSynchronize(c->stream));
  if (norm_prev_host) *norm_prev_host = sc.prev_norm;
  if (t_host) *t_host = (int64_t)sc.t;
  return FIRA_OK;
}

fira_status fira_set_state(fira_ctx* c, int32_t idx, const float* M_dev, const float* V_dev, float norm_prev,
                           int64_t t) {
  fira_status s = check_idx(c, idx); if (s != FIRA_OK) return s;
  if (t < 0 || isnan(norm_prev)) { set_error("t must be >= 0 and norm_prev not NaN"); return FIRA_ERR_INVALID_ARG; }
  const MatDev& mt = c->mats[idx];
  const size_t bytes = (size_t)mt.l * mt.r * 4;
  if (M_dev) FIRA_CUDA(cudaMemcpyAsync(mt.M, M_dev, bytes, cudaMemcpyDeviceToDevice, c->stream));
  if (V_dev) FIRA_CUDA(cudaMemcpyAsync(mt.V, V_dev, bytes, cudaMemcpyDeviceToDevice, c->stream));
  MatScalars sc;
  memset(&sc, 0, sizeof(sc));
  sc.prev_norm = norm_prev < 0.f ? -1.f : norm_prev;
  sc.lambda = 1.f;
  sc.t = t;
  FIRA_CUDA(cudaMemcpyAsync(mt.sc, &sc, sizeof(sc), cudaMemcpyHostToDevice, c->stream));
  FIRA_CUDA(cudaStreamSynchronize(c->stream));
  c->t_host[idx] = t;
  return FIRA_OK;
}

int64_t fira_state_elements(const fira_ctx* c, int32_t idx) {
  if (!c || idx < 0 || idx >= (int)c->mats.size()) return -1;
  const MatDev& mt = c->mats[idx];
  return (int64_t)mt.d * mt.r + 2 * (int64_t)mt.l * mt.r + 1;
}

fira_status fira_get_diagnostics(fira_ctx* c, int32_t idx, fira_diag* out) {
  fira_status s = check_idx(c, idx); if (s != FIRA_OK) return s;
  if (!out) { set_error("null output pointer"); return FIRA_ERR_INVALID_ARG; }
  MatScalars sc;
  FIRA_CUDA(cudaMemcpyAsync(&sc, c->mats[idx].sc, sizeof(sc), cudaMemcpyDeviceToHost, c->stream));
  FIRA_CUDA(cudaStreamSynchronize(c->stream));
  out->norm_scaled = sc.norm_scaled; out->lambda = sc.lambda; out->norm_prev = sc.prev_norm;
  out->k_min = sc.k_min; out->k_max = sc.k_max; out->t = (int64_t)sc.t;
  out->engine = c->mats[idx].engine;
  return FIRA_OK;
}

fira_status fira_poll(fira_ctx* c) {
  if (!c) { set_error("null context"); return FIRA_ERR_INVALID_ARG; }
  unsigned st = 0;
  FIRA_CUDA(cudaMemcpyAsync(&st, c->status_dev, sizeof(st), cudaMemcpyDeviceToHost, c->stream));
  FIRA_CUDA(cudaStreamSynchronize(c->stream));
  if (st != 0) FIRA_CUDA(cudaMemsetAsync(c->status_dev, 0, sizeof(unsigned), c->stream));
  if (st & DEV_STATUS_TIMEOUT) { set_error("a bounded device-side wait ran out"); return FIRA_ERR_DEVICE_TIMEOUT; }
  if (st & DEV_STATUS_NONFINITE) { set_error("a non-finite norm or factor was produced"); return FIRA_ERR_NONFINITE; }
  return FIRA_OK;
}

fira_status fira_selftest_bounded_wait(fira_ctx* c, int32_t rounds) {
  if (!c) { set_error("null context"); return FIRA_ERR_INVALID_ARG; }
  if (rounds < 1 || rounds > (1 << 20)) { set_error("rounds must lie in [1, 2^20]"); return FIRA_ERR_INVALID_ARG; }
  return tc_selftest_bounded_wait(c, rounds);
}

int32_t fira_last_step_launches(const fira_ctx* c) { return c ? c->last_launches : -1; }

fira_status fira_enable_phase_timing(fira_ctx* c, int32_t enable) {
  if (!c) { set_error("null context"); return FIRA_ERR_INVALID_ARG; }
  PhaseTimer& tm = c->timer;
  if (enable && tm.events.empty()) {
    tm.events.resize((size_t)FIRA_TIMING_MAX_STEPS * (FIRA_TIMING_MAX_PHASES + 1));
    for (auto& ev : tm.events) FIRA_CUDA(cudaEventCreate(&ev));
    if (c->simt.nlist) for (int i = 0; i < 6; ++i) tm.names.push_back(kSimtPhaseNames[i]);
    if (!c->tc_list.empty()) {
      const char* nm[8];
      const int k = tc_phase_names(nm);
      for (int i = 0; i < k; ++i) tm.names.push_back(nm[i]);
    }
  }
  tm.on = enable != 0;
  tm.steps = 0;
  return FIRA_OK;
}

fira_status fira_get_phase_times(fira_ctx* c, int32_t* nphases, float* ms_out, int32_t* steps_recorded) {
  if (!c || !nphases || !ms_out || !steps_recorded) { set_error("null argument"); return FIRA_ERR_INVALID_ARG; }
  PhaseTimer& tm = c->timer;
  FIRA_CUDA(cudaStreamSynchronize(c->stream));
  const int np = (int)tm.names.size();
  const int ns = (int)std::min<long long>(tm.steps, FIRA_TIMING_MAX_STEPS);
  *nphases = np; *steps_recorded = ns;
  for (int p = 0; p < np; ++p) {
    double acc = 0.0;
    for (int s = 0; s < ns; ++s) {
      float ms = 0.f;
      const size_t base = (size_t)s * (FIRA_TIMING_MAX_PHASES + 1);
      FIRA_CUDA(cudaEventElapsedTime(&ms, tm.events[base + p], tm.events[base + p + 1]));
      acc += ms;
    }
    ms_out[p] = ns ? (float)(acc / ns) : 0.f;
  }
  return FIRA_OK;
}

const char* fira_phase_name(const fira_ctx* c, int32_t phase) {
  if (!c || phase < 0 || phase >= (int)c->timer.names.size()) return "";
  return c->timer.names[phase];
}

const char* fira_status_string(fira_status s) {
  switch (s) {
    case FIRA_OK: return "ok";
    case FIRA_ERR_INVALID_ARG: return "invalid argument";
    case FIRA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case FIRA_ERR_UNSUPPORTED: return "unsupported";
    case FIRA_ERR_CUDA: return "CUDA error";
    case FIRA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case FIRA_ERR_NONFINITE: return "non-finite value";
  }
  return "unknown status";
}

const char* fira_last_error(void) { return g_last_error.c_str(); }

void fira_destroy(fira_ctx* c) {
  if (!c) return;
  tc_destroy_plan(c);
  if (c->pipe.in) {
    cudaStreamDestroy(c->pipe.in); cudaStreamDestroy(c->pipe.out);
    cudaEventDestroy(c->pipe.start); cudaEventDestroy(c->pipe.out_done);
    for (auto& ev : c->pipe.in_done) cudaEventDestroy(ev);
    for (auto& ev : c->pipe.stepped) cudaEventDestroy(ev);
  }
  for (auto& ev : c->timer.events) cudaEventDestroy(ev);
  delete c;
}

}  // extern "C"
