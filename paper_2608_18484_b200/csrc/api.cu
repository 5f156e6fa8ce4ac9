// C-ABI layer: argument validation, workspace carving, launch order.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>
#include "kernels.cuh"

using namespace spr;

namespace spr {
int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); return 148; }
    cached[dev] = n;
  }
  return cached[dev];
}
}  // namespace spr

namespace {

struct Carver {                       // bump allocator over a caller-owned workspace (or a dry run)
  char* base;
  size_t off = 0;
  explicit Carver(void* b) : base(static_cast<char*>(b)) {}
  template <typename T> T* take(size_t n) {
    off = (off + 255) & ~size_t(255);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
  size_t bytes() const { return (off + 255) & ~size_t(255); }
};

struct Resolved {
  int B, H, BH, N, d, dtype, es;
  int Hkv, G, BHkv;                    // K/V heads, query heads per K/V head (1 = ordinary multi-head attention), B * Hkv
  int Ck, Cq, Cmax, Ms, M, rK, rQ, RK, RQ, Rmax, r_out, T, mode;
  int partition;                       // sparsepr_partition_t
  int fK, fQ;                          // width of the features each side is clustered in: rK / rQ, or d for raw activations
  bool full_rank;                      // r_out covers the whole row space of the probe residuals: the projector is the identity
  float density, lambda, eps_rms, eps_std, scale;
  u64 seed;
  int head_offset;                 // first head of this call within the whole problem (keys the row samples)
  i64 qs[3], ks[3], vs[3], os[3];
};

int round16(int r) { return feature_ld(r); }      // row length of a feature buffer with r columns

sparsepr_status_t resolve(const sparsepr_shape_t* s, const sparsepr_params_t* p, Resolved* r) {
  if (!s || !r) return SPARSEPR_ERR_INVALID_ARG;
  if (s->B < 1 || s->H < 1 || s->N < 1) return SPARSEPR_ERR_INVALID_ARG;
  if (s->dtype != SPARSEPR_F32 && s->dtype != SPARSEPR_BF16) return SPARSEPR_ERR_INVALID_ARG;
  if ((s->d != 64 && s->d != 128) || s->dv != s->d) return SPARSEPR_ERR_UNSUPPORTED;
  r->B = s->B; r->H = s->H; r->BH = s->B * s->H; r->N = s->N; r->d = s->d; r->dtype = s->dtype;
  r->Hkv = s->Hkv > 0 ? s->Hkv : s->H;
  if (s->Hkv < 0 || r->Hkv > s->H || s->H % r->Hkv != 0) return SPARSEPR_ERR_INVALID_ARG;
  r->G = s->H / r->Hkv; r->BHkv = s->B * r->Hkv;
  // grouped-query attention runs on the tensor-core kernels only
  if (r->G > 1 && !(s->dtype == SPARSEPR_BF16 && s->d == 128)) return SPARSEPR_ERR_UNSUPPORTED;
  r->es = s->dtype == SPARSEPR_BF16 ? 2 : 4;
  const int vec = 16 / r->es;
  for (int i = 0; i < 3; ++i) {
    r->qs[i] = s->q_stride[i]; r->ks[i] = s->k_stride[i]; r->vs[i] = s->v_stride[i]; r->os[i] = s->o_stride[i];
    if (r->qs[i] < 0 || r->ks[i] < 0 || r->vs[i] < 0 || r->os[i] < 0) return SPARSEPR_ERR_INVALID_ARG;
    if (r->qs[i] % vec || r->ks[i] % vec || r->vs[i] % vec || r->os[i] % vec) return SPARSEPR_ERR_UNSUPPORTED;
  }
  if (r->qs[2] < s->d || r->ks[2] < s->d || r->vs[2] < s->d || r->os[2] < s->d) return SPARSEPR_ERR_INVALID_ARG;
  if (!p) return SPARSEPR_OK;
  if (!(p->density > 0.f) || p->block < 0 || p->Ck < 0 || p->Cq < 0 || p->n_sample < 0 || p->n_probe < 0 ||
      p->rK < 0 || p->rQ < 0 || p->r_out < 0 || p->kmeans_iters < 0 || p->mode < 0 || p->mode > 1 ||
      !(p->softmax_scale >= 0.f) || !(p->eps_rms >= 0.f) || !(p->eps_std >= 0.f) || std::isnan(p->lambda))
    return SPARSEPR_ERR_INVALID_ARG;
  const int block = p->block ? p->block : 128;
  r->Ck = p->Ck ? p->Ck : (s->N + block - 1) / block;
  r->Cq = p->Cq ? p->Cq : (s->N + block - 1) / block;
  if (r->Ck > s->N || r->Cq > s->N) return SPARSEPR_ERR_INVALID_ARG;
  if (r->Ck > kMaxGroups || r->Cq > kMaxGroups) return SPARSEPR_ERR_UNSUPPORTED;
  r->Cmax = r->Ck > r->Cq ? r->Ck : r->Cq;
  r->Ms = std::min(p->n_sample ? p->n_sample : 256, s->N);
  r->mode = p->mode;
  r->M = r->mode == 1 ? 0 : std::min(p->n_probe, s->N);
  if (r->M > kMaxProbes) return SPARSEPR_ERR_UNSUPPORTED;
  r->rK = std::min(p->rK ? p->rK : 48, s->d);
  r->rQ = std::min(p->rQ ? p->rQ : 64, s->d);
  if (r->rK > kMaxRank || r->rQ > kMaxRank) return SPARSEPR_ERR_UNSUPPORTED;
  if (p->partition < 0 || p->partition > SPARSEPR_PARTITION_SEMANTIC) return SPARSEPR_ERR_INVALID_ARG;
  r->partition = p->partition;
  r->fK = r->partition == SPARSEPR_PARTITION_SEMANTIC ? s->d : r->rK;
  r->fQ = r->partition != SPARSEPR_PARTITION_RESPONSE_COUPLED ? s->d : r->rQ;
  r->RK = round16(r->fK); r->RQ = round16(r->fQ); r->Rmax = std::max(r->RK, r->RQ);
  {
    // r = min(r_out, M, d_v).  Once r reaches min(M, d_v) it spans every direction the probe residuals (M rows in
    // d_v dimensions) can have, the projector acts as the identity and no eigenvectors are needed; below that the
    // eigen-solver delivers at most kMaxRank of them.
    const int want = p->r_out ? p->r_out : 16, cap = std::min(std::max(r->M, 1), s->d);
    r->full_rank = want >= cap;
    r->r_out = std::max(1, std::min(want, cap));
    if (!r->full_rank && r->r_out > kMaxRank) return SPARSEPR_ERR_UNSUPPORTED;
  }
  r->T = p->kmeans_iters ? p->kmeans_iters : 8;
  r->density = p->density;
  r->lambda = p->lambda < 0.f ? 0.1f : p->lambda;
  r->eps_rms = p->eps_rms > 0.f ? p->eps_rms : 1e-6f;
  r->eps_std = p->eps_std > 0.f ? p->eps_std : 1e-6f;
  r->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / std::sqrt((float)s->d);
  r->seed = p->seed;
  if (p->head_offset < 0 || p->head_offset % r->G != 0) return SPARSEPR_ERR_INVALID_ARG;
  r->head_offset = p->head_offset;
  return SPARSEPR_OK;
}

std::once_flag g_init_once;
cudaError_t g_init_err = cudaSuccess;
cudaError_t ensure_init() {
  std::call_once(g_init_once, [] {
    cudaError_t e;
    if ((e = init_eigen()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_group_sort()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_routing()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_attention_simt()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_attention_tc()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_correction_tc()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_attention_packed()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_project_tc()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_kmeans_tc()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_probe_tc()) != cudaSuccess) { g_init_err = e; return; }
    if ((e = init_fit()) != cudaSuccess) { g_init_err = e; return; }
  });
  return g_init_err;
}

bool launch_ok() {
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess && std::getenv("SPARSEPR_DEBUG")) std::fprintf(stderr, "sparsepr: CUDA error: %s\n", cudaGetErrorString(e));
  return e == cudaSuccess;
}

// Optional per-stage CUDA-event timing of one call.  Events are recorded on the call's
// stream between stages; finish() synchronises once and accumulates the elapsed times.
struct StageTimer {
  sparsepr_profile_t* out;
  cudaStream_t st;
  std::vector<cudaEvent_t> ev;
  std::vector<int> stage;
  StageTimer(sparsepr_profile_t* o, cudaStream_t s) : out(o), st(s) { mark(-1); }
  void mark(int stage_done) {
    if (!out) return;
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) { out = nullptr; return; }
    cudaEventRecord(e, st);
    ev.push_back(e);
    stage.push_back(stage_done);
  }
  void finish() {
    if (out && !ev.empty() && cudaEventSynchronize(ev.back()) == cudaSuccess) {
      for (size_t i = 1; i < ev.size(); ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ev[i - 1], ev[i]) == cudaSuccess && stage[i] >= 0 && stage[i] < SPARSEPR_STAGE_COUNT)
          out->ms[stage[i]] += ms;
      }
    }
    for (cudaEvent_t e : ev) cudaEventDestroy(e);
    ev.clear();
  }
};

}  // namespace

// Auxiliary streams and events of one plan.  They are created once and recycled: a plan takes a set from a
// per-process pool (keyed by device) and hands it back when it is destroyed, so that a steady stream of calls
// creates nothing.  A set belongs to one plan at a time, hence concurrent calls never share an event.
struct SideSet {
  int device = -1;
  // second stream for work that is independent of the main chain (probe selection next to routing;
  // probe rows and fit next to the block-sparse kernel), forked and joined with the two events
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // third stream: the remainder kernel beside the 128-row kernel
  cudaStream_t side2 = nullptr;
  cudaEvent_t ev_join2 = nullptr;
};
namespace {
std::mutex g_side_mu;
std::vector<SideSet*> g_side_pool;

SideSet* acquire_side_set() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  {
    std::lock_guard<std::mutex> lk(g_side_mu);
    for (size_t i = 0; i < g_side_pool.size(); ++i)
      if (g_side_pool[i]->device == dev) {
        SideSet* s = g_side_pool[i];
        g_side_pool.erase(g_side_pool.begin() + i);
        return s;
      }
  }
  SideSet* s = new (std::nothrow) SideSet();
  if (!s) return nullptr;
  s->device = dev;
  int prio_lo = 0, prio_hi = 0;
  cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
  if (cudaStreamCreateWithPriority(&s->side, cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
      cudaStreamCreateWithPriority(&s->side2, cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
      cudaEventCreateWithFlags(&s->ev_join2, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&s->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&s->ev_join, cudaEventDisableTiming) != cudaSuccess) {
    if (s->ev_fork) cudaEventDestroy(s->ev_fork);
    if (s->ev_join) cudaEventDestroy(s->ev_join);
    if (s->ev_join2) cudaEventDestroy(s->ev_join2);
    if (s->side) cudaStreamDestroy(s->side);
    if (s->side2) cudaStreamDestroy(s->side2);
    delete s;
    return nullptr;
  }
  return s;
}
void release_side_set(SideSet* s) {
  if (!s) return;
  std::lock_guard<std::mutex> lk(g_side_mu);
  g_side_pool.push_back(s);
}
}  // namespace

struct sparsepr_plan_s {
  Resolved r;
  cudaStream_t stream;
  SideSet* set = nullptr;
  cudaStream_t side = nullptr, side2 = nullptr;          // aliases of the set's members
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_join2 = nullptr;
  // the probe selection of the plan call may still run on `side` when the call returns: the first attend call
  // orders it (its probe work follows on the same stream and is joined there); statistics, export and the
  // destructor wait for it themselves
  mutable bool side_pending = false;
  bool imported = false;                                  // built by sparsepr_plan_import: no partition stages ran
  ~sparsepr_plan_s() {
    if (side && side_pending) cudaStreamSynchronize(side);
    release_side_set(set);
  }
  // device state (all inside the caller's plan workspace)
  int* err; int* recheck;
  double* Mmat; double* lam;
  float *FK, *FQ, *phi;
  unsigned* maxabs; int* fx_shift;
  float *mu, *mu2, *mumax; i64* sums; int* counts;
  int *a_K, *a_Q, *kv_perm, *kv_inv, *q_perm, *q_inv, *kv_off, *q_off, *nk, *nq;
  float *kappa, *theta, *score;
  int *route_ptr, *route_idx, *tile_off, *tile_off128;
  RouteState* rstate;
  double* probe_dist; int* probe_idx; float* probe_w;
  __nv_bfloat16 *xh, *xl, *mh, *ml, *Ft; float* xnorm; int* flagged; int* flagcnt; double* eigws;
  int *rem_pos, *rem_grp, *rem_cnt;      // rows of the short group remainders (packed attention tiles)
  int* km_changed;                       // [2 sides][T + 1][BH] rows that changed group in each k-means pass
  double* Mpool;                         // [BHkv][d][d] key-response metric pooled over the query heads of a K/V head (grouped-query attention only)
};

namespace {

void carve_plan(Carver& c, const Resolved& r, sparsepr_plan_s* p) {
  const size_t BH = r.BH, N = r.N, d = r.d;
  int* err = c.take<int>(64);
  int* recheck = err ? err + 1 : nullptr;
  double* Mmat = c.take<double>(BH * d * d);
  double* lam = c.take<double>(BH * d);
  float* FK = c.take<float>(BH * d * r.rK);
  float* FQ = c.take<float>(BH * d * r.rQ);
  float* phi = c.take<float>(BH * N * r.Rmax);
  unsigned* maxabs = c.take<unsigned>(BH);
  int* fx = c.take<int>(BH);
  float* mu = c.take<float>(BH * r.Cmax * r.Rmax);
  float* mu2 = c.take<float>(BH * r.Cmax);
  float* mumax = c.take<float>(BH);
  i64* sums = c.take<i64>(BH * r.Cmax * r.Rmax);
  int* counts = c.take<int>(BH * r.Cmax);
  int* aK = c.take<int>(BH * N); int* aQ = c.take<int>(BH * N);
  int* kvp = c.take<int>(BH * N); int* kvi = c.take<int>(BH * N);
  int* qp = c.take<int>(BH * N); int* qi = c.take<int>(BH * N);
  int* kvo = c.take<int>(BH * (r.Ck + 1)); int* qo = c.take<int>(BH * (r.Cq + 1));
  int* nk = c.take<int>(BH * r.Ck); int* nq = c.take<int>(BH * r.Cq);
  float* kappa = c.take<float>(BH * r.Ck * d); float* theta = c.take<float>(BH * r.Cq * d);
  float* score = c.take<float>(BH * (size_t)r.Cq * r.Ck);
  int* rptr = c.take<int>(BH * (r.Cq + 1)); int* ridx = c.take<int>(BH * (size_t)r.Cq * r.Ck);
  int* toff = c.take<int>(BH * (r.Cq + 1));
  int* toff128 = c.take<int>(BH * (r.Cq + 1));
  RouteState* rs = c.take<RouteState>(BH);
  double* pd = c.take<double>(BH * N);
  int* pidx = c.take<int>(BH * std::max(r.M, 1)); float* pw = c.take<float>(BH * std::max(r.M, 1));
  __nv_bfloat16* xh = c.take<__nv_bfloat16>(BH * N * 64); __nv_bfloat16* xl = c.take<__nv_bfloat16>(BH * N * 64);
  __nv_bfloat16* mh = c.take<__nv_bfloat16>(BH * (size_t)r.Cmax * 64); __nv_bfloat16* ml = c.take<__nv_bfloat16>(BH * (size_t)r.Cmax * 64);
  float* xnorm = c.take<float>(BH * N); int* flagged = c.take<int>(BH * N);
  __nv_bfloat16* Ft = c.take<__nv_bfloat16>(BH * (size_t)3 * 64 * 128);
  int* rem_pos = c.take<int>(BH * N); int* rem_grp = c.take<int>(BH * N); int* rem_cnt = c.take<int>(BH);
  int* km_changed = c.take<int>(2 * (size_t)(r.T + 1) * BH);
  int* flagcnt = c.take<int>(2 * BH);                       // two sets of per-head counters, used by alternate passes
  double* eigws = c.take<double>(eig_scratch_doubles((int)BH, r.d));
  double* Mpool = c.take<double>(r.G > 1 ? (size_t)r.BHkv * d * d : 0);
  if (p) {
    p->km_changed = km_changed; p->flagcnt = flagcnt; p->eigws = eigws; p->Mpool = Mpool; p->Ft = Ft; p->rem_pos = rem_pos; p->rem_grp = rem_grp; p->rem_cnt = rem_cnt;
    p->err = err; p->recheck = recheck; p->Mmat = Mmat; p->lam = lam; p->FK = FK; p->FQ = FQ; p->phi = phi;
    p->maxabs = maxabs; p->fx_shift = fx; p->mu = mu; p->mu2 = mu2; p->mumax = mumax; p->sums = sums; p->counts = counts;
    p->a_K = aK; p->a_Q = aQ; p->kv_perm = kvp; p->kv_inv = kvi; p->q_perm = qp; p->q_inv = qi; p->kv_off = kvo; p->q_off = qo;
    p->nk = nk; p->nq = nq; p->kappa = kappa; p->theta = theta; p->score = score; p->route_ptr = rptr; p->route_idx = ridx;
    p->xh = xh; p->xl = xl; p->mh = mh; p->ml = ml; p->xnorm = xnorm; p->flagged = flagged;
    p->tile_off = toff; p->tile_off128 = toff128; p->rstate = rs; p->probe_dist = pd; p->probe_idx = pidx; p->probe_w = pw;
  }
}

struct AttendWs {
  void *Qg, *Kg, *Vg;
  __nv_bfloat16* Olo;                  // second bf16 word of the hard-drop rows for the correction pass (tensor-core path, fitted mode)
  float *partial, *X, *Dn, *A, *c, *Psi;
  __nv_bfloat16 *At, *Qp;
  int n_split_tc;
  double* fit; double* fit_eigws;
  int n_split;
};

int probe_splits(const Resolved& r) {
  if (r.M == 0) return 1;
  const int row_tiles = (r.M + 63) / 64;
  int s = (2 * sm_count() + r.BH * row_tiles - 1) / (r.BH * row_tiles);
  const int key_tiles = (r.N + 63) / 64;
  s = std::max(1, std::min(s, std::max(1, key_tiles / 4)));
  return s;
}

void carve_attend(Carver& c, const Resolved& r, AttendWs* w) {
  const size_t BH = r.BH, N = r.N, d = r.d;
  const int ns = probe_splits(r);
  void* Qg = c.take<char>(BH * N * d * r.es);
  void* Kg = c.take<char>(BH * N * d * r.es);
  void* Vg = c.take<char>(BH * N * d * r.es);
  const bool staged = r.dtype == SPARSEPR_BF16 && r.d == 128 && r.mode == 0 && r.M > 0;
  __nv_bfloat16* Olo = c.take<__nv_bfloat16>(staged ? BH * N * d : 0);
  const size_t M1 = std::max(r.M, 1);
  // tensor-core probe kernel: one CTA per (128 probe rows, key slice), about one wave
  const int ns_tc = std::max(1, std::min(sm_count() / std::max(1, r.BH * (int)((M1 + 127) / 128)), std::max(1, r.N / 128 / 4)));
  float* partial = c.take<float>(probe_partial_floats(r.BH, std::max(ns, ns_tc), (int)M1, r.d));
  __nv_bfloat16* Qp = c.take<__nv_bfloat16>(BH * M1 * d);
  float* X = c.take<float>(BH * M1 * d); float* Dn = c.take<float>(BH * M1 * d);
  float* A = c.take<float>(BH * d * d); float* cc = c.take<float>(BH * d);
  float* Psi = c.take<float>(BH * d * d);
  __nv_bfloat16* At = c.take<__nv_bfloat16>(2 * BH * d * d);   // the correction map as two bf16 words
  double* fit = c.take<double>(fit_scratch_doubles(r.BH, (int)M1, r.d));
  double* fit_eigws = c.take<double>(eig_scratch_doubles(r.BH, r.d));
  if (w) { w->Olo = Olo; w->Qg = Qg; w->Kg = Kg; w->Vg = Vg; w->partial = partial; w->X = X; w->Dn = Dn; w->A = A; w->c = cc; w->Psi = Psi; w->At = At; w->Qp = Qp; w->n_split_tc = ns_tc; w->fit = fit; w->fit_eigws = fit_eigws; w->n_split = ns; }
}

i64 pair_budget(const Resolved& r) {
  const i64 total = (i64)std::floor((double)r.density * (double)r.N * (double)r.N);
  return std::max<i64>(total - (i64)r.M * r.N, 0);
}

void run_kmeans(const sparsepr_plan_s* p, int r, int C, int tag, int* assign, const int* warm_prev, int nheads, cudaStream_t st) {
  const Resolved& R = p->r;
  const int ld = round16(r);
  // changed[t][bh], t = 1..T: rows of head bh that changed group in pass t.  A pass that changes nothing proves the
  // fixed point, so the later passes of that head return at once (their result would be identical).
  int* changed = p->km_changed + (tag == kTagQInit ? (size_t)(R.T + 1) * R.BH : 0);
  cudaMemsetAsync(changed, 0, (size_t)(R.T + 1) * R.BH * sizeof(int), st);
  launch_kmeans_init(p->phi, ld, nheads, R.N, r, C, R.seed, tag, tag == kTagQInit ? R.head_offset : R.head_offset / R.G, p->mu, p->sums, p->counts, p->maxabs, p->fx_shift, st);
  const bool tcp = kmeans_tc_supported() && r <= kMaxRank;
  float* mumax = tcp ? nullptr : p->mumax;       // the tensor-core assignment derives the norm bound from ||mu||^2 itself
  // (with the tensor-core assignment the finalize step also writes the two bf16 words of every centroid)
  // warm start: the initial centroids become the means of the current features over the previous partition's groups
  if (warm_prev) launch_kmeans_warm_sums(p->phi, ld, nheads, R.N, r, C, warm_prev, p->sums, p->counts, p->fx_shift, st);
  launch_kmeans_finalize(p->mu, p->mu2, mumax, p->sums, p->counts, p->fx_shift, nheads, C, r, warm_prev ? 1 : 0, st, tcp ? p->mh : nullptr, tcp ? p->ml : nullptr);
  if (tcp) launch_split_bf16(p->phi, ld, (i64)nheads * R.N, r, p->xh, p->xl, p->xnorm, st);
  if (tcp) cudaMemsetAsync(p->flagcnt, 0, 2 * (size_t)R.BH * sizeof(int), st);
  for (int t = 1; t <= R.T; ++t) {
    const bool upd = t < R.T;
    const int* prev = t > 1 ? changed + (size_t)(t - 1) * R.BH : nullptr;
    int* cur = changed + (size_t)t * R.BH;
    if (tcp) {
      KmeansTcArgs ka{};
      ka.BH = nheads; ka.N = R.N; ka.C = C; ka.r = r; ka.R = ld; ka.xh = p->xh; ka.xl = p->xl; ka.mh = p->mh; ka.ml = p->ml;
      ka.phi = p->phi; ka.ldphi = ld; ka.xnorm = p->xnorm; ka.mu = p->mu; ka.mu2 = p->mu2;
      ka.assign = assign; ka.sums = upd ? p->sums : nullptr; ka.counts = upd ? p->counts : nullptr; ka.fx_shift = p->fx_shift;
      ka.flagged = p->flagged; ka.flag_count = p->flagcnt + (size_t)(t & 1) * R.BH; ka.flag_count_next = p->flagcnt + (size_t)((t + 1) & 1) * R.BH;
      ka.recheck_total = p->recheck; ka.err = p->err;
      ka.prev_changed = prev; ka.cur_changed = cur;
      launch_kmeans_assign_tc(ka, st);
    } else {
      if (!upd) cudaMemsetAsync(p->recheck, 0, sizeof(int), st);
      launch_kmeans_assign(p->phi, ld, nheads, R.N, r, p->mu, p->mu2, p->mumax, C, assign, upd ? p->sums : nullptr,
                           upd ? p->counts : nullptr, p->fx_shift, p->recheck, prev, cur, st);
    }
    if (upd) launch_kmeans_finalize(p->mu, p->mu2, mumax, p->sums, p->counts, p->fx_shift, nheads, C, r, 1, st, tcp ? p->mh : nullptr, tcp ? p->ml : nullptr);
  }
}

// pads [n][r] rows to [n][R] with zeros
__global__ void k_pad_rows(const float* __restrict__ in, int n, int r, int R, float* __restrict__ out) {
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < (i64)n * R; e += (i64)gridDim.x * blockDim.x) {
    const int k = (int)(e % R);
    out[e] = k < r ? in[(e / R) * r + k] : 0.f;
  }
}
// key-response metric of a K/V head = mean of the sampled-query second moments of its G query heads
__global__ void k_pool_metric(const double* __restrict__ Mq, int G, int dd, double* __restrict__ out) {
  const int kvh = blockIdx.y;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < dd; e += gridDim.x * blockDim.x) {
    double s = 0.0;
    for (int g = 0; g < G; ++g) s += Mq[((i64)kvh * G + g) * dd + e];
    out[(i64)kvh * dd + e] = s / (double)G;
  }
}
__global__ void k_sizes_from_off(const int* __restrict__ off, int C, int* __restrict__ sizes) {
  const int bh = blockIdx.y;
  for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < C; g += gridDim.x * blockDim.x)
    sizes[(i64)bh * C + g] = off[(i64)bh * (C + 1) + g + 1] - off[(i64)bh * (C + 1) + g];
}

}  // namespace

extern "C" {

const char* sparsepr_status_string(sparsepr_status_t s) {
  switch (s) {
    case SPARSEPR_OK: return "ok";
    case SPARSEPR_ERR_INVALID_ARG: return "invalid argument";
    case SPARSEPR_ERR_UNSUPPORTED: return "unsupported shape or parameter";
    case SPARSEPR_ERR_WORKSPACE: return "workspace too small or misaligned";
    case SPARSEPR_ERR_CUDA: return "CUDA error";
    case SPARSEPR_ERR_NUMERIC: return "numerical breakdown or non-finite input";
    case SPARSEPR_ERR_TIMEOUT: return "bounded device wait ran out";
  }
  return "unknown status";
}

size_t sparsepr_plan_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params) {
  Resolved r;
  if (!params || resolve(shape, params, &r) != SPARSEPR_OK) return 0;
  Carver c(nullptr);
  carve_plan(c, r, nullptr);
  return c.bytes();
}

size_t sparsepr_attend_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params) {
  Resolved r;
  if (!params || resolve(shape, params, &r) != SPARSEPR_OK) return 0;
  Carver c(nullptr);
  carve_attend(c, r, nullptr);
  return c.bytes();
}

static sparsepr_status_t make_plan(const sparsepr_shape_t* shape, const sparsepr_params_t* params, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream, sparsepr_plan_s** out) {
  if (!params || !out) return SPARSEPR_ERR_INVALID_ARG;
  Resolved r;
  sparsepr_status_t s = resolve(shape, params, &r);
  if (s != SPARSEPR_OK) return s;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SPARSEPR_ERR_WORKSPACE;
  Carver dry(nullptr);
  carve_plan(dry, r, nullptr);
  if (workspace_bytes < dry.bytes()) return SPARSEPR_ERR_WORKSPACE;
  if (ensure_init() != cudaSuccess) return SPARSEPR_ERR_CUDA;
  sparsepr_plan_s* p = new (std::nothrow) sparsepr_plan_s();
  if (!p) return SPARSEPR_ERR_INVALID_ARG;
  p->r = r;
  p->stream = static_cast<cudaStream_t>(cuda_stream);
  p->set = acquire_side_set();
  if (!p->set) { delete p; return SPARSEPR_ERR_CUDA; }
  p->side = p->set->side; p->side2 = p->set->side2;
  p->ev_fork = p->set->ev_fork; p->ev_join = p->set->ev_join; p->ev_join2 = p->set->ev_join2;
  Carver c(workspace);
  carve_plan(c, r, p);
  *out = p;
  return SPARSEPR_OK;
}

// the side stream starts after everything queued on `st` so far ...
void fork_side(const sparsepr_plan_s* p, cudaStream_t st) {
  cudaEventRecord(p->ev_fork, st);
  cudaStreamWaitEvent(p->side, p->ev_fork, 0);
}
// ... and `st` continues once the side stream's work is done
void join_side(const sparsepr_plan_s* p, cudaStream_t st) {
  cudaEventRecord(p->ev_join, p->side);
  cudaStreamWaitEvent(st, p->ev_join, 0);
}

static sparsepr_status_t plan_impl(const sparsepr_shape_t* shape, const sparsepr_params_t* params, const void* Q,
                                   const void* K, void* workspace, size_t workspace_bytes, void* cuda_stream,
                                   sparsepr_plan_t** out, sparsepr_profile_t* prof, const int* warm_kv = nullptr,
                                   const int* warm_q = nullptr) {
  if (!Q || !K) return SPARSEPR_ERR_INVALID_ARG;
  sparsepr_plan_s* p = nullptr;
  sparsepr_status_t s = make_plan(shape, params, workspace, workspace_bytes, cuda_stream, &p);
  if (s != SPARSEPR_OK) return s;
  const Resolved& r = p->r;
  // grouped-query attention shares feature maps and K/V copies between heads: tensor-core kernels only
  if (r.G > 1 && !(kmeans_tc_supported() && project_tc_supported(r.dtype, r.d, r.rQ, r.qs) && project_tc_supported(r.dtype, r.d, r.rK, r.ks))) {
    delete p;
    return SPARSEPR_ERR_UNSUPPORTED;
  }
  cudaStream_t st = p->stream;
  cudaGetLastError();
  cudaMemsetAsync(p->err, 0, 64 * sizeof(int), st);
  cudaMemsetAsync(p->maxabs, 0, r.BH * sizeof(unsigned), st);
  StageTimer tm(prof, st);
  // K/V partition: sampled-query metric -> F_K -> phi_K -> k-means (semantic variant: k-means on K itself)
  if (r.partition == SPARSEPR_PARTITION_SEMANTIC) {
    tm.mark(SPARSEPR_STAGE_KEY_METRIC);
    launch_raw_features(r.dtype, K, r.ks, r.BHkv, r.Hkv, r.N, r.d, p->phi, p->maxabs, p->err, st);
  } else {
    // every query head samples its own rows; under grouped-query attention the K/V head's metric is the mean over its
    // query heads (Section 4.3: the K/V partition is shared by the associated query heads)
    launch_sample_gram(r.dtype, Q, r.qs, r.BH, r.H, r.N, r.d, r.Ms, r.seed, r.head_offset, p->Mmat, st);
    const double* metric = p->Mmat;
    if (r.G > 1) {
      k_pool_metric<<<dim3(16, r.BHkv), 256, 0, st>>>(p->Mmat, r.G, r.d * r.d, p->Mpool);
      metric = p->Mpool;
    }
    launch_eig_top(metric, (i64)r.d * r.d, r.BHkv, r.d, r.rK, 0, r.dtype == SPARSEPR_F32, p->FK, p->lam, p->eigws, st);
    tm.mark(SPARSEPR_STAGE_KEY_METRIC);
    if (project_tc_supported(r.dtype, r.d, r.rK, r.ks)) {
      if (!launch_project_tc(K, r.ks, r.BHkv, r.Hkv, r.N, r.rK, p->FK, false, 0.f, p->phi, r.RK, p->maxabs, p->Ft, p->err, st)) { delete p; return SPARSEPR_ERR_CUDA; }
    } else {
      launch_project(r.dtype, K, r.ks, r.BHkv, r.Hkv, r.N, r.d, r.rK, p->FK, false, 0.f, p->phi, r.RK, p->maxabs, p->err, st);
    }
  }
  tm.mark(SPARSEPR_STAGE_KEY_PROJECT);
  run_kmeans(p, r.fK, r.Ck, kTagKvInit, p->a_K, warm_kv, r.BHkv, st);
  tm.mark(SPARSEPR_STAGE_KEY_KMEANS);
  launch_group_sort(p->a_K, r.BHkv, r.N, r.Ck, p->kv_perm, p->kv_inv, p->kv_off, p->err, st);
  launch_group_means(r.dtype, K, r.ks, r.BHkv, r.Hkv, p->kv_perm, p->kv_off, r.N, r.Ck, r.d, p->kappa, p->nk, st);
  tm.mark(SPARSEPR_STAGE_KEY_PERMUTE);
  // query partition: centroid metric -> F_Q -> phi_Q -> k-means (other variants: k-means on Q itself)
  cudaMemsetAsync(p->maxabs, 0, r.BH * sizeof(unsigned), st);
  if (r.partition != SPARSEPR_PARTITION_RESPONSE_COUPLED) {
    tm.mark(SPARSEPR_STAGE_QUERY_METRIC);
    launch_raw_features(r.dtype, Q, r.qs, r.BH, r.H, r.N, r.d, p->phi, p->maxabs, p->err, st);
  } else {
    launch_centroid_gram(p->kappa, p->nk, r.BHkv, r.Ck, r.d, p->Mmat, st);
    launch_eig_top(p->Mmat, (i64)r.d * r.d, r.BHkv, r.d, r.rQ, 0, r.dtype == SPARSEPR_F32, p->FQ, p->lam, p->eigws, st);
    tm.mark(SPARSEPR_STAGE_QUERY_METRIC);
    if (project_tc_supported(r.dtype, r.d, r.rQ, r.qs)) {
      if (!launch_project_tc(Q, r.qs, r.BH, r.H, r.N, r.rQ, p->FQ, true, r.eps_rms, p->phi, r.RQ, p->maxabs, p->Ft, p->err, st, r.G)) { delete p; return SPARSEPR_ERR_CUDA; }
    } else {
      launch_project(r.dtype, Q, r.qs, r.BH, r.H, r.N, r.d, r.rQ, p->FQ, true, r.eps_rms, p->phi, r.RQ, p->maxabs, p->err, st);
    }
  }
  tm.mark(SPARSEPR_STAGE_QUERY_PROJECT);
  run_kmeans(p, r.fQ, r.Cq, kTagQInit, p->a_Q, warm_q, r.BH, st);
  tm.mark(SPARSEPR_STAGE_QUERY_KMEANS);
  launch_group_sort(p->a_Q, r.BH, r.N, r.Cq, p->q_perm, p->q_inv, p->q_off, p->err, st);
  launch_group_means(r.dtype, Q, r.qs, r.BH, r.H, p->q_perm, p->q_off, r.N, r.Cq, r.d, p->theta, p->nq, st);
  tm.mark(SPARSEPR_STAGE_QUERY_PERMUTE);
  // probes and routes; without a profile the probe selection runs beside the routing
  const bool overlap = prof == nullptr && r.M > 0;
  cudaStream_t ps = st;
  if (overlap) { fork_side(p, st); ps = p->side; }
  if (r.M > 0)
    launch_probe_select(p->phi, r.RQ, r.fQ, p->q_perm, p->q_off, p->nq, r.BH, r.N, r.Cq, r.M, p->probe_dist, p->probe_idx, p->probe_w, ps);
  tm.mark(SPARSEPR_STAGE_PROBE_SELECT);
  launch_cell_scores(p->theta, p->kappa, p->nq, p->nk, r.BH, r.Cq, r.Ck, r.d, r.scale, p->score, r.G, st);
  launch_route_select(p->score, p->nq, p->nk, r.BH, r.Cq, r.Ck, pair_budget(r), r.density >= 1.0f, p->route_ptr,
                      p->route_idx, p->rstate, nullptr, r.G, st);
  launch_tile_offsets(p->q_off, r.BH, r.Cq, 64, 0, p->tile_off, st);
  launch_tile_offsets(p->q_off, r.BH, r.Cq, 128, kRemRows, p->tile_off128, st);
  launch_remainder_rows(p->q_off, p->route_ptr, p->route_idx, r.BH, r.Cq, r.Ck, r.N, p->rem_pos, p->rem_grp, p->rem_cnt, st);
  if (overlap) p->side_pending = true;          // not joined here: the probes are not needed before the attend call
  tm.mark(SPARSEPR_STAGE_ROUTE);
  tm.finish();
  if (!launch_ok()) { delete p; return SPARSEPR_ERR_CUDA; }
  *out = p;
  return SPARSEPR_OK;
}

sparsepr_status_t sparsepr_plan(const sparsepr_shape_t* shape, const sparsepr_params_t* params, const void* Q,
                                const void* K, const void* V, void* workspace, size_t workspace_bytes,
                                void* cuda_stream, sparsepr_plan_t** out) {
  (void)V;
  return plan_impl(shape, params, Q, K, workspace, workspace_bytes, cuda_stream, out, nullptr);
}

sparsepr_status_t sparsepr_plan_timed(const sparsepr_shape_t* shape, const sparsepr_params_t* params, const void* Q,
                                      const void* K, const void* V, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream, sparsepr_plan_t** out, sparsepr_profile_t* profile) {
  (void)V;
  if (!profile) return SPARSEPR_ERR_INVALID_ARG;
  return plan_impl(shape, params, Q, K, workspace, workspace_bytes, cuda_stream, out, profile);
}

sparsepr_status_t sparsepr_plan_warm(const sparsepr_shape_t* shape, const sparsepr_params_t* params, const void* Q,
                                     const void* K, const void* V, const int32_t* prev_kv_assign,
                                     const int32_t* prev_q_assign, void* workspace, size_t workspace_bytes,
                                     void* cuda_stream, sparsepr_plan_t** out) {
  (void)V;
  if (!prev_kv_assign || !prev_q_assign) return SPARSEPR_ERR_INVALID_ARG;
  return plan_impl(shape, params, Q, K, workspace, workspace_bytes, cuda_stream, out, nullptr, prev_kv_assign, prev_q_assign);
}

sparsepr_status_t sparsepr_plan_assignments(const sparsepr_plan_t* p, const int32_t** kv_assign, const int32_t** q_assign) {
  if (!p || !kv_assign || !q_assign) return SPARSEPR_ERR_INVALID_ARG;
  *kv_assign = p->a_K;
  *q_assign = p->a_Q;
  return SPARSEPR_OK;
}

sparsepr_status_t sparsepr_plan_import(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                       const sparsepr_plan_host_t* in, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream, sparsepr_plan_t** out) {
  if (!in || !in->kv_assign || !in->q_assign || !in->route_ptr || !in->route_idx) return SPARSEPR_ERR_INVALID_ARG;
  sparsepr_plan_s* p = nullptr;
  sparsepr_status_t s = make_plan(shape, params, workspace, workspace_bytes, cuda_stream, &p);
  if (s != SPARSEPR_OK) return s;
  const Resolved& r = p->r;
  if (r.M > 0 && (!in->probe_idx || !in->probe_w)) { delete p; return SPARSEPR_ERR_INVALID_ARG; }
  p->imported = true;
  cudaStream_t st = p->stream;
  cudaGetLastError();
  const size_t BH = r.BH, N = r.N;
  cudaMemsetAsync(p->err, 0, 64 * sizeof(int), st);
  cudaMemcpyAsync(p->a_K, in->kv_assign, (size_t)r.BHkv * N * sizeof(int), cudaMemcpyHostToDevice, st);
  cudaMemcpyAsync(p->a_Q, in->q_assign, BH * N * sizeof(int), cudaMemcpyHostToDevice, st);
  cudaMemcpyAsync(p->route_ptr, in->route_ptr, BH * (r.Cq + 1) * sizeof(int), cudaMemcpyHostToDevice, st);
  cudaMemcpyAsync(p->route_idx, in->route_idx, BH * (size_t)r.Cq * r.Ck * sizeof(int), cudaMemcpyHostToDevice, st);
  if (r.M > 0) {
    cudaMemcpyAsync(p->probe_idx, in->probe_idx, BH * r.M * sizeof(int), cudaMemcpyHostToDevice, st);
    cudaMemcpyAsync(p->probe_w, in->probe_w, BH * r.M * sizeof(float), cudaMemcpyHostToDevice, st);
  }
  launch_group_sort(p->a_K, r.BHkv, r.N, r.Ck, p->kv_perm, p->kv_inv, p->kv_off, p->err, st);
  launch_group_sort(p->a_Q, r.BH, r.N, r.Cq, p->q_perm, p->q_inv, p->q_off, p->err, st);
  k_sizes_from_off<<<dim3((r.Ck + 255) / 256, r.BHkv), 256, 0, st>>>(p->kv_off, r.Ck, p->nk);
  k_sizes_from_off<<<dim3((r.Cq + 255) / 256, r.BH), 256, 0, st>>>(p->q_off, r.Cq, p->nq);
  launch_count_pairs(p->q_off, p->kv_off, p->route_ptr, p->route_idx, r.BH, r.Cq, r.Ck, p->rstate, r.G, st);
  launch_tile_offsets(p->q_off, r.BH, r.Cq, 64, 0, p->tile_off, st);
  launch_tile_offsets(p->q_off, r.BH, r.Cq, 128, kRemRows, p->tile_off128, st);
  launch_remainder_rows(p->q_off, p->route_ptr, p->route_idx, r.BH, r.Cq, r.Ck, r.N, p->rem_pos, p->rem_grp, p->rem_cnt, st);
  if (!launch_ok() || cudaStreamSynchronize(st) != cudaSuccess) { delete p; return SPARSEPR_ERR_CUDA; }
  *out = p;
  return SPARSEPR_OK;
}

void sparsepr_plan_destroy(sparsepr_plan_t* plan) { delete plan; }

static sparsepr_status_t attend_impl(const sparsepr_plan_t* p, const void* Q, const void* K, const void* V, void* O,
                                     float* O_sparse, void* workspace, size_t workspace_bytes, void* cuda_stream,
                                     sparsepr_profile_t* prof) {
  if (!p || !Q || !K || !V || !O) return SPARSEPR_ERR_INVALID_ARG;
  const Resolved& r = p->r;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SPARSEPR_ERR_WORKSPACE;
  Carver dry(nullptr);
  carve_attend(dry, r, nullptr);
  if (workspace_bytes < dry.bytes()) return SPARSEPR_ERR_WORKSPACE;
  AttendWs w;
  Carver c(workspace);
  carve_attend(c, r, &w);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaGetLastError();
  StageTimer tm(prof, st);
  launch_gather_rows(r.dtype, Q, r.qs, r.BH, r.H, p->q_perm, r.N, r.d, w.Qg, st);
  launch_gather_rows(r.dtype, K, r.ks, r.BHkv, r.Hkv, p->kv_perm, r.N, r.d, w.Kg, st);
  launch_gather_rows(r.dtype, V, r.vs, r.BHkv, r.Hkv, p->kv_perm, r.N, r.d, w.Vg, st);
  tm.mark(SPARSEPR_STAGE_GATHER);
  const bool fitted = r.mode == 0 && r.M > 0;
  AttnArgs aa{};
  aa.dtype = r.dtype; aa.BH = r.BH; aa.H = r.H; aa.N = r.N; aa.d = r.d; aa.scale = r.scale;
  aa.Q = w.Qg; aa.K = w.Kg; aa.V = w.Vg;
  aa.q_off = p->q_off; aa.kv_off = p->kv_off; aa.route_ptr = p->route_ptr; aa.route_idx = p->route_idx;
  aa.q_perm = p->q_perm; aa.tile_off = p->tile_off; aa.Cq = r.Cq; aa.Ck = r.Ck; aa.kv_div = r.G;
  aa.O = O; for (int i = 0; i < 3; ++i) aa.os[i] = r.os[i];
  aa.O_sparse = O_sparse;
  aa.err = p->err;
  const bool tensor = attention_tc_supported(aa);
  // The probe rows and the fit depend only on the gathered K, V and the plan.  With the tensor-core
  // kernel (whose correction is a separate pass) they run on the plan's second stream beside the
  // block-sparse kernel; a profiled call keeps everything on one stream so that stage times add up.
  const bool overlap = fitted && tensor && prof == nullptr;
  if (p->side_pending && !overlap) { join_side(p, st); p->side_pending = false; }   // the plan call's probe selection, still on the second stream
  if (fitted) {
    cudaStream_t fs = st;
    if (overlap) { fork_side(p, st); fs = p->side; }
    ProbeArgs pa{};
    pa.dtype = r.dtype; pa.BH = r.BH; pa.H = r.H; pa.N = r.N; pa.d = r.d; pa.M = r.M; pa.Ck = r.Ck; pa.Cq = r.Cq;
    pa.n_split = w.n_split; pa.scale = r.scale; pa.Q = Q; pa.kv_div = r.G;
    for (int i = 0; i < 3; ++i) pa.qs[i] = r.qs[i];
    pa.Kg = w.Kg; pa.Vg = w.Vg; pa.probe_idx = p->probe_idx; pa.q_assign = p->a_Q; pa.kv_off = p->kv_off;
    pa.route_ptr = p->route_ptr; pa.route_idx = p->route_idx; pa.partial = w.partial; pa.X = w.X; pa.Dn = w.Dn;
    if (probe_tc_supported(pa)) {
      pa.n_split = w.n_split_tc;
      if (!launch_probe_rows_tc(pa, w.Qp, p->err, fs)) return SPARSEPR_ERR_CUDA;
      launch_probe_merge(pa, fs);
    } else {
      launch_probe_rows(pa, fs);
    }
    tm.mark(SPARSEPR_STAGE_PROBE_ROWS);
    FitArgs fa{};
    fa.BH = r.BH; fa.M = r.M; fa.d = r.d; fa.r_out = r.r_out; fa.full_rank = r.full_rank; fa.lambda = r.lambda; fa.eps_std = r.eps_std; fa.precise = r.dtype == SPARSEPR_F32;
    fa.X = w.X; fa.Dn = w.Dn; fa.w = p->probe_w; fa.scratch = w.fit; fa.eig_ws = w.fit_eigws; fa.A = w.A; fa.c = w.c; fa.Psi = w.Psi; fa.err = p->err;
    launch_fit(fa, fs);
    tm.mark(SPARSEPR_STAGE_FIT);
  }
  if (tensor) {
    aa.tile_off = p->tile_off128;
    // with a correction to follow, the block-sparse kernels also store what the bf16 rounding of O dropped
    if (fitted) aa.O_lo = w.Olo;
    // the packed remainder tiles are few and long, the 128-row tiles many and short: they share the GPU instead of
    // running one after the other (also in a profiled call: both belong to the ATTENTION stage)
    if (!overlap) cudaEventRecord(p->ev_fork, st);                // (with the probes' overlap the event is recorded already)
    cudaStreamWaitEvent(p->side2, p->ev_fork, 0);
    if (!launch_attention_packed(aa, p->rem_pos, p->rem_grp, p->rem_cnt, p->side2)) return SPARSEPR_ERR_CUDA;
    if (!launch_attention_tc(aa, st)) return SPARSEPR_ERR_CUDA;
    cudaEventRecord(p->ev_join2, p->side2);
    cudaStreamWaitEvent(st, p->ev_join2, 0);
    tm.mark(SPARSEPR_STAGE_ATTENTION);
    if (overlap) { join_side(p, st); p->side_pending = false; }
    if (fitted && !launch_correction_tc(w.A, w.c, w.At, w.Olo, O, r.os, r.BH, r.H, r.N, p->err, st)) return SPARSEPR_ERR_CUDA;
    tm.mark(SPARSEPR_STAGE_CORRECTION);
  } else {
    aa.A = fitted ? w.A : nullptr; aa.c = fitted ? w.c : nullptr;      // correction fused into this kernel's epilogue
    launch_attention_simt(aa, st);
    tm.mark(SPARSEPR_STAGE_ATTENTION);
  }
  if (fitted) launch_write_probe_rows(r.dtype, w.Dn, p->probe_idx, r.BH, r.H, r.M, r.d, O, r.os, st);
  tm.mark(SPARSEPR_STAGE_PROBE_WRITE);
  tm.finish();
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_attend(const sparsepr_plan_t* p, const void* Q, const void* K, const void* V, void* O,
                                  float* O_sparse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return attend_impl(p, Q, K, V, O, O_sparse, workspace, workspace_bytes, cuda_stream, nullptr);
}

sparsepr_status_t sparsepr_attend_timed(const sparsepr_plan_t* p, const void* Q, const void* K, const void* V, void* O,
                                        float* O_sparse, void* workspace, size_t workspace_bytes, void* cuda_stream,
                                        sparsepr_profile_t* profile) {
  if (!profile) return SPARSEPR_ERR_INVALID_ARG;
  return attend_impl(p, Q, K, V, O, O_sparse, workspace, workspace_bytes, cuda_stream, profile);
}

sparsepr_status_t sparsepr_dense_timed(const sparsepr_shape_t* shape, float softmax_scale, const void* Q, const void* K,
                                       const void* V, void* O, void* cuda_stream, sparsepr_profile_t* profile) {
  if (!profile) return SPARSEPR_ERR_INVALID_ARG;
  StageTimer tm(profile, static_cast<cudaStream_t>(cuda_stream));
  sparsepr_status_t s = sparsepr_dense(shape, softmax_scale, Q, K, V, O, cuda_stream);
  tm.mark(SPARSEPR_STAGE_DENSE);
  tm.finish();
  return s;
}

sparsepr_status_t sparsepr_dense(const sparsepr_shape_t* shape, float softmax_scale, const void* Q, const void* K,
                                 const void* V, void* O, void* cuda_stream) {
  if (!Q || !K || !V || !O) return SPARSEPR_ERR_INVALID_ARG;
  Resolved r;
  sparsepr_status_t s = resolve(shape, nullptr, &r);
  if (s != SPARSEPR_OK) return s;
  if (!(softmax_scale >= 0.f)) return SPARSEPR_ERR_INVALID_ARG;
  if (ensure_init() != cudaSuccess) return SPARSEPR_ERR_CUDA;
  cudaGetLastError();
  AttnArgs aa{};
  aa.dtype = r.dtype; aa.BH = r.BH; aa.H = r.H; aa.N = r.N; aa.d = r.d; aa.kv_div = r.G;
  aa.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt((float)r.d);
  aa.Q = Q; aa.K = K; aa.V = V; aa.O = O;
  for (int i = 0; i < 3; ++i) { aa.qs[i] = r.qs[i]; aa.ks[i] = r.ks[i]; aa.vs[i] = r.vs[i]; aa.os[i] = r.os[i]; }
  if (attention_tc_supported(aa)) {
    if (!launch_attention_tc(aa, static_cast<cudaStream_t>(cuda_stream))) return SPARSEPR_ERR_CUDA;
  } else {
    launch_attention_simt(aa, static_cast<cudaStream_t>(cuda_stream));
  }
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_plan_device_error(const sparsepr_plan_t* p, int32_t* device_error) {
  if (!p || !device_error) return SPARSEPR_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess || (p->side && cudaStreamSynchronize(p->side) != cudaSuccess)) return SPARSEPR_ERR_CUDA;
  int errw = 0;
  if (cudaMemcpy(&errw, p->err, sizeof(errw), cudaMemcpyDeviceToHost) != cudaSuccess) return SPARSEPR_ERR_CUDA;
  *device_error = errw;
  return SPARSEPR_OK;
}

sparsepr_status_t sparsepr_plan_stats(const sparsepr_plan_t* p, sparsepr_stats_t* out) {
  if (!p || !out) return SPARSEPR_ERR_INVALID_ARG;
  const Resolved& r = p->r;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess || (p->side && cudaStreamSynchronize(p->side) != cudaSuccess)) return SPARSEPR_ERR_CUDA;
  std::memset(out, 0, sizeof(*out));
  std::vector<RouteState> rs(r.BH);
  std::vector<int> qo((size_t)r.BH * (r.Cq + 1)), ko((size_t)r.BHkv * (r.Ck + 1)), rp((size_t)r.BH * (r.Cq + 1));
  std::vector<int> ri((size_t)r.BH * r.Cq * r.Ck);
  int errw[2] = {0, 0};
  if (cudaMemcpy(rs.data(), p->rstate, rs.size() * sizeof(RouteState), cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(qo.data(), p->q_off, qo.size() * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(ko.data(), p->kv_off, ko.size() * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(rp.data(), p->route_ptr, rp.size() * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(ri.data(), p->route_idx, ri.size() * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemcpy(errw, p->err, sizeof(errw), cudaMemcpyDeviceToHost) != cudaSuccess)
    return SPARSEPR_ERR_CUDA;
  out->rho_route_min = 1e300; out->rho_route_max = -1.0;
  out->nonempty_kv_groups_min = r.Ck; out->nonempty_q_groups_min = r.Cq;
  const double nn = (double)r.N * (double)r.N;
  for (int bh = 0; bh < r.BH; ++bh) {
    out->routed_pairs += rs[bh].pairs;
    out->routed_cells += rs[bh].cells;
    const double rho = (double)rs[bh].pairs / nn;
    out->rho_route += rho / r.BH;
    out->rho_route_min = std::min(out->rho_route_min, rho);
    out->rho_route_max = std::max(out->rho_route_max, rho);
    int neK = 0, neQ = 0;
    const int* k = &ko[(size_t)(bh / r.G) * (r.Ck + 1)];
    const int* q = &qo[(size_t)bh * (r.Cq + 1)];
    for (int g = 0; g < r.Ck; ++g) { neK += k[g + 1] > k[g]; out->max_kv_group = std::max(out->max_kv_group, k[g + 1] - k[g]); }
    for (int g = 0; g < r.Cq; ++g) { neQ += q[g + 1] > q[g]; out->max_q_group = std::max(out->max_q_group, q[g + 1] - q[g]); }
    out->nonempty_kv_groups_min = std::min(out->nonempty_kv_groups_min, neK);
    out->nonempty_q_groups_min = std::min(out->nonempty_q_groups_min, neQ);
    // pairs issued by the tiled kernel over the concatenated routed keys: the tensor-core kernel uses
    // 128-row query tiles and 128-key tiles built from 16-row boxes, the float32 kernel 64 x 64 tiles
    const bool tcpath = r.dtype == SPARSEPR_BF16 && r.d == 128;
    const int qtile = tcpath ? 128 : 64, ktile = tcpath ? 128 : 64, box = tcpath ? 16 : 1;
    const int* rpp = &rp[(size_t)bh * (r.Cq + 1)];
    const int* rii = &ri[(size_t)bh * r.Cq * r.Ck];
    // packed tiles: 128 remainder rows each, groups in the order of k_remainder_rows (routed groups descending, first
    // route ascending, id); a tile streams the union of the K/V groups its rows route to
    std::vector<char> want(r.Ck, 0);
    int packed_fill = 0;
    auto flush_packed = [&]() {
      i64 boxes = 0;
      for (int g = 0; g < r.Ck; ++g) if (want[g]) { boxes += (k[g + 1] - k[g] + box - 1) / box; want[g] = 0; }
      out->padded_tile_pairs += (i64)qtile * ((boxes * box + ktile - 1) / ktile) * ktile;
      packed_fill = 0;
    };
    std::vector<unsigned long long> packed_order;
    for (int a = 0; a < r.Cq; ++a) {
      i64 keys = 0;
      for (int t = rpp[a]; t < rpp[a + 1]; ++t) keys += (k[rii[t] + 1] - k[rii[t]] + box - 1) / box * box;
      const i64 kt = (keys + ktile - 1) / ktile;
      const int nrow = q[a + 1] - q[a], rem = nrow % qtile;
      if (tcpath && rem > 0 && rem <= kRemRows) {
        // full tiles by the 128-row kernel; the short remainder joins the packed tiles
        out->padded_tile_pairs += (i64)(nrow / qtile) * qtile * kt * ktile;
        const int n = rpp[a + 1] - rpp[a];
        packed_order.push_back(((unsigned long long)(r.Ck - n) << 24) | ((unsigned long long)(n > 0 ? rii[rpp[a]] : 0) << 12) | (unsigned long long)a);
      } else {
        out->padded_tile_pairs += (i64)((nrow + qtile - 1) / qtile) * qtile * kt * ktile;
      }
    }
    std::sort(packed_order.begin(), packed_order.end());
    for (unsigned long long key : packed_order) {
      const int a = (int)(key & 0xFFFull);
      for (int left = (q[a + 1] - q[a]) % qtile; left > 0;) {
        const int take = std::min(left, qtile - packed_fill);
        for (int t = rpp[a]; t < rpp[a + 1]; ++t) want[rii[t]] = 1;
        packed_fill += take; left -= take;
        if (packed_fill == qtile) flush_packed();
      }
    }
    if (packed_fill > 0) flush_packed();
  }
  out->rho_exec = out->rho_route + (double)r.M / (double)r.N;
  out->assign_rechecked_rows = errw[1];
  out->device_error = errw[0];
  // k-means passes that ran before every head had reached its fixed point (or T)
  std::vector<int> ch(2 * (size_t)(r.T + 1) * r.BH);
  if (cudaMemcpy(ch.data(), p->km_changed, ch.size() * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SPARSEPR_ERR_CUDA;
  for (int side = 0; side < 2 && !p->imported; ++side) {
    int worst = 0;
    for (int bh = 0; bh < (side == 0 ? r.BHkv : r.BH); ++bh) {
      int ran = 1;
      while (ran < r.T && ch[((size_t)side * (r.T + 1) + ran) * r.BH + bh] > 0) ++ran;
      worst = std::max(worst, ran);
    }
    (side == 0 ? out->kmeans_passes_kv : out->kmeans_passes_q) = worst;
  }
  return SPARSEPR_OK;
}

sparsepr_status_t sparsepr_plan_export(const sparsepr_plan_t* p, sparsepr_plan_host_t* o) {
  if (!p || !o) return SPARSEPR_ERR_INVALID_ARG;
  const Resolved& r = p->r;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess || (p->side && cudaStreamSynchronize(p->side) != cudaSuccess)) return SPARSEPR_ERR_CUDA;
  const size_t BH = r.BH, N = r.N;
  bool ok = true;
  auto cp = [&](void* dst, const void* src, size_t bytes) { if (dst && bytes) ok &= cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost) == cudaSuccess; };
  const size_t BHkv = r.BHkv;
  cp(o->kv_assign, p->a_K, BHkv * N * 4); cp(o->q_assign, p->a_Q, BH * N * 4);
  cp(o->kv_perm, p->kv_perm, BHkv * N * 4); cp(o->q_perm, p->q_perm, BH * N * 4);
  cp(o->kv_off, p->kv_off, BHkv * (r.Ck + 1) * 4); cp(o->q_off, p->q_off, BH * (r.Cq + 1) * 4);
  cp(o->route_ptr, p->route_ptr, BH * (r.Cq + 1) * 4); cp(o->route_idx, p->route_idx, BH * (size_t)r.Cq * r.Ck * 4);
  cp(o->probe_idx, p->probe_idx, BH * r.M * 4); cp(o->probe_w, p->probe_w, BH * r.M * 4);
  if (o->routed_pairs) {
    std::vector<RouteState> rs(BH);
    cp(rs.data(), p->rstate, BH * sizeof(RouteState));
    for (size_t i = 0; i < BH; ++i) o->routed_pairs[i] = rs[i].pairs;
  }
  return ok ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_plan_export_features(const sparsepr_plan_t* p, sparsepr_plan_features_t* o) {
  if (!p || !o) return SPARSEPR_ERR_INVALID_ARG;
  if (p->imported) return SPARSEPR_ERR_UNSUPPORTED;          // an imported plan never computed them
  const Resolved& r = p->r;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess || (p->side && cudaStreamSynchronize(p->side) != cudaSuccess)) return SPARSEPR_ERR_CUDA;
  const size_t BH = r.BH, N = r.N, d = r.d;
  bool ok = true;
  auto cp = [&](void* dst, const void* src, size_t bytes) { if (dst && bytes) ok &= cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost) == cudaSuccess; };
  const size_t BHkv = r.BHkv;
  if (r.partition != SPARSEPR_PARTITION_SEMANTIC) cp(o->F_K, p->FK, BHkv * d * r.rK * 4);
  if (r.partition == SPARSEPR_PARTITION_RESPONSE_COUPLED) cp(o->F_Q, p->FQ, BHkv * d * r.rQ * 4);
  if (o->phi_Q)                                                // rows are padded to RQ floats on the device
    ok &= cudaMemcpy2D(o->phi_Q, (size_t)r.fQ * 4, p->phi, (size_t)r.RQ * 4, (size_t)r.fQ * 4, BH * N, cudaMemcpyDeviceToHost) == cudaSuccess;
  cp(o->kappa, p->kappa, BHkv * r.Ck * d * 4); cp(o->theta, p->theta, BH * r.Cq * d * 4);
  cp(o->score, p->score, BH * (size_t)r.Cq * r.Ck * 4);
  return ok ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_selftest_bounded_wait(int32_t* device_error_word, void* cuda_stream) {
  if (!device_error_word) return SPARSEPR_ERR_INVALID_ARG;
  cudaGetLastError();
  launch_selftest_bounded_wait(device_error_word, static_cast<cudaStream_t>(cuda_stream));
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

// ---- single stages ---------------------------------------------------------------------
size_t sparsepr_stage_assign_workspace_bytes(int32_t n, int32_t C, int32_t r) {
  if (n < 1 || C < 1 || r < 1 || r > kMaxRank) return 0;
  const size_t R = round16(r);
  Carver c(nullptr);
  c.take<float>((size_t)n * R); c.take<float>((size_t)C * R); c.take<float>(C); c.take<float>(1); c.take<int>(4);
  c.take<__nv_bfloat16>((size_t)n * 64); c.take<__nv_bfloat16>((size_t)n * 64);
  c.take<__nv_bfloat16>((size_t)C * 64); c.take<__nv_bfloat16>((size_t)C * 64); c.take<float>(n); c.take<int>(n);
  return c.bytes();
}

sparsepr_status_t sparsepr_stage_assign(int32_t n, int32_t C, int32_t r, const float* X, const float* mu, int32_t* a,
                                        void* ws, size_t ws_bytes, void* cuda_stream) {
  if (n < 1 || C < 1 || r < 1 || !X || !mu || !a) return SPARSEPR_ERR_INVALID_ARG;
  if (r > kMaxRank) return SPARSEPR_ERR_UNSUPPORTED;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) || ws_bytes < sparsepr_stage_assign_workspace_bytes(n, C, r))
    return SPARSEPR_ERR_WORKSPACE;
  if (ensure_init() != cudaSuccess) return SPARSEPR_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int R = round16(r);
  Carver c(ws);
  float* Xp = c.take<float>((size_t)n * R); float* mup = c.take<float>((size_t)C * R);
  float* mu2 = c.take<float>(C); float* mumax = c.take<float>(1); int* fx = c.take<int>(4);
  __nv_bfloat16* xh = c.take<__nv_bfloat16>((size_t)n * 64); __nv_bfloat16* xl = c.take<__nv_bfloat16>((size_t)n * 64);
  __nv_bfloat16* mh = c.take<__nv_bfloat16>((size_t)C * 64); __nv_bfloat16* ml = c.take<__nv_bfloat16>((size_t)C * 64);
  float* xnorm = c.take<float>(n); int* flagged = c.take<int>(n);
  cudaGetLastError();
  k_pad_rows<<<(unsigned)std::min<i64>(((i64)n * R + 255) / 256, 65535), 256, 0, st>>>(X, n, r, R, Xp);
  k_pad_rows<<<(unsigned)std::min<i64>(((i64)C * R + 255) / 256, 65535), 256, 0, st>>>(mu, C, r, R, mup);
  launch_kmeans_finalize(mup, mu2, mumax, nullptr, nullptr, fx, 1, C, r, 0, st);
  if (kmeans_tc_supported() && C <= kMaxGroups) {
    launch_split_bf16(Xp, R, n, r, xh, xl, xnorm, st);
    launch_split_bf16(mup, R, C, r, mh, ml, nullptr, st);
    KmeansTcArgs ka{};
    ka.BH = 1; ka.N = n; ka.C = C; ka.r = r; ka.R = R; ka.xh = xh; ka.xl = xl; ka.mh = mh; ka.ml = ml;
    ka.phi = Xp; ka.ldphi = R; ka.xnorm = xnorm; ka.mu = mup; ka.mu2 = mu2; ka.assign = a;
    ka.flagged = flagged; ka.flag_count = fx + 1; ka.recheck_total = fx + 2;
    cudaMemsetAsync(ka.flag_count, 0, sizeof(int), st);
    if (!launch_kmeans_assign_tc(ka, st)) return SPARSEPR_ERR_CUDA;
  } else {
    launch_kmeans_assign(Xp, R, 1, n, r, mup, mu2, mumax, C, a, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, st);
  }
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_stage_permute(int32_t n, int32_t C, const int32_t* a, int32_t* perm, int32_t* inv,
                                         int32_t* off, void* cuda_stream) {
  if (n < 1 || C < 1 || !a || !perm || !inv || !off) return SPARSEPR_ERR_INVALID_ARG;
  if (C > kMaxGroups) return SPARSEPR_ERR_UNSUPPORTED;
  if (ensure_init() != cudaSuccess) return SPARSEPR_ERR_CUDA;
  cudaGetLastError();
  launch_group_sort(a, 1, n, C, perm, inv, off, nullptr, static_cast<cudaStream_t>(cuda_stream));
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

sparsepr_status_t sparsepr_stage_route(int32_t Cq, int32_t Ck, const float* score, const int32_t* nq, const int32_t* nk,
                                       int64_t pair_budget, int32_t select_all, int32_t* route_ptr, int32_t* route_idx,
                                       int64_t* pairs_out, void* cuda_stream) {
  if (Cq < 1 || Ck < 1 || !score || !nq || !nk || !route_ptr || !route_idx || !pairs_out) return SPARSEPR_ERR_INVALID_ARG;
  if (Cq > kMaxGroups || Ck > kMaxGroups) return SPARSEPR_ERR_UNSUPPORTED;
  if (ensure_init() != cudaSuccess) return SPARSEPR_ERR_CUDA;
  cudaGetLastError();
  launch_route_select(score, nq, nk, 1, Cq, Ck, pair_budget, select_all, route_ptr, route_idx, nullptr, reinterpret_cast<i64*>(pairs_out),
                      1, static_cast<cudaStream_t>(cuda_stream));
  return launch_ok() ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
}

}  // extern "C"
