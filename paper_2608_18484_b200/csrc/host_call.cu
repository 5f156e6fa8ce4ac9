// sparsepr_call_host: a whole SparsePR call for tensors in host memory, as a pipeline over groups of heads.
//
// Heads are independent (Section 4.3 shares only the K/V partition inside a group of query heads), so a problem
// can be cut into groups of consecutive heads.  One stream uploads group after group, two streams take the groups
// in turn through sparsepr_plan + sparsepr_attend (the latency-bound stages of one group run beside the attention
// kernel of the other), a fourth stream returns every group's output.  A group runs with head_offset = its first
// head, which keeps the deterministic row samples (Appendix B.1; k-means initialisation) those of one call over all
// heads.  Everything here goes through the public entry points; the file holds no arithmetic of the method.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "sparsepr.h"

namespace {

struct Box { int b0, b1, h0, h1; };

// Groups of consecutive heads (order b H + h): whole batch entries when there are at least `groups` of them,
// otherwise ranges of K/V heads (with their query heads) inside each batch entry.
std::vector<Box> head_groups(int B, int H, int Hkv, int groups) {
  std::vector<Box> out;
  const int G = H / Hkv;
  groups = std::max(1, std::min(groups, B * Hkv));
  if (B >= groups) {
    for (int i = 0; i < groups; ++i) {
      const int b0 = (int)((long long)B * i / groups), b1 = (int)((long long)B * (i + 1) / groups);
      if (b1 > b0) out.push_back({b0, b1, 0, H});
    }
    return out;
  }
  const int per_b = std::max(1, std::min((groups + B - 1) / B, Hkv));
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < per_b; ++i) {
      const int h0 = (int)((long long)Hkv * i / per_b) * G, h1 = (int)((long long)Hkv * (i + 1) / per_b) * G;
      if (h1 > h0) out.push_back({b, b + 1, h0, h1});
    }
  return out;
}

// Streams and events of one call in flight, recycled through a per-process pool (keyed by device).
struct Pipe {
  int device = -1;
  cudaStream_t up = nullptr, down = nullptr, work = nullptr;
  std::vector<cudaEvent_t> ev;
  bool grow(size_t n) {
    while (ev.size() < n) {
      cudaEvent_t e;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return false;
      ev.push_back(e);
    }
    return true;
  }
};
std::mutex g_pipe_mu;
std::vector<Pipe*> g_pipe_pool;

Pipe* acquire_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  {
    std::lock_guard<std::mutex> lk(g_pipe_mu);
    for (size_t i = 0; i < g_pipe_pool.size(); ++i)
      if (g_pipe_pool[i]->device == dev) {
        Pipe* p = g_pipe_pool[i];
        g_pipe_pool.erase(g_pipe_pool.begin() + i);
        return p;
      }
  }
  Pipe* p = new (std::nothrow) Pipe();
  if (!p) return nullptr;
  p->device = dev;
  if (cudaStreamCreateWithFlags(&p->up, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&p->down, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&p->work, cudaStreamNonBlocking) != cudaSuccess) {
    if (p->up) cudaStreamDestroy(p->up);
    if (p->down) cudaStreamDestroy(p->down);
    if (p->work) cudaStreamDestroy(p->work);
    delete p;
    return nullptr;
  }
  return p;
}
void release_pipe(Pipe* p) {
  if (!p) return;
  std::lock_guard<std::mutex> lk(g_pipe_mu);
  g_pipe_pool.push_back(p);
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Shape of one group inside the contiguous device copies of the whole problem.
sparsepr_shape_t sub_shape(const sparsepr_shape_t& s, int Hkv, const Box& b) {
  sparsepr_shape_t t = s;
  const int G = s.H / Hkv;
  t.B = b.b1 - b.b0;
  t.H = b.h1 - b.h0;
  t.Hkv = (b.h1 - b.h0) / G;
  const long long nd = (long long)s.N * s.d;
  const long long qs[3] = {(long long)s.H * nd, nd, s.d}, ks[3] = {(long long)Hkv * nd, nd, s.d};
  for (int i = 0; i < 3; ++i) { t.q_stride[i] = qs[i]; t.o_stride[i] = qs[i]; t.k_stride[i] = ks[i]; t.v_stride[i] = ks[i]; }
  return t;
}

struct Layout {
  size_t es, nq, nk;                  // element size, bytes of Q (= O), bytes of K (= V)
  size_t q, k, v, o;                  // offsets of the device copies
  std::vector<size_t> plan_off, plan_bytes, att_off, att_bytes;
  size_t total = 0;
};

bool lay_out(const sparsepr_shape_t* shape, const sparsepr_params_t* params, int groups, std::vector<Box>* boxes,
             Layout* L) {
  if (!shape || !params) return false;
  if (shape->B < 1 || shape->H < 1 || shape->N < 1 || shape->d < 1) return false;
  const int Hkv = shape->Hkv > 0 ? shape->Hkv : shape->H;
  if (Hkv > shape->H || shape->H % Hkv != 0) return false;
  if (params->head_offset < 0) return false;
  L->es = shape->dtype == SPARSEPR_F32 ? 4 : 2;
  const size_t nd = (size_t)shape->N * shape->d;
  L->nq = (size_t)shape->B * shape->H * nd * L->es;
  L->nk = (size_t)shape->B * Hkv * nd * L->es;
  size_t off = 0;
  L->q = off; off += align256(L->nq);
  L->k = off; off += align256(L->nk);
  L->v = off; off += align256(L->nk);
  L->o = off; off += align256(L->nq);
  *boxes = head_groups(shape->B, shape->H, Hkv, groups < 1 ? 4 : groups);
  for (const Box& b : *boxes) {
    const sparsepr_shape_t t = sub_shape(*shape, Hkv, b);
    sparsepr_params_t p = *params;
    p.head_offset = params->head_offset + b.b0 * shape->H + b.h0;
    const size_t pb = sparsepr_plan_workspace_bytes(&t, &p), ab = sparsepr_attend_workspace_bytes(&t, &p);
    if (pb == 0 || ab == 0) return false;
    L->plan_off.push_back(off); L->plan_bytes.push_back(pb); off += align256(pb);
    L->att_off.push_back(off); L->att_bytes.push_back(ab); off += align256(ab);
  }
  L->total = off;
  return true;
}

}  // namespace

extern "C" {

int32_t sparsepr_head_groups(int32_t B, int32_t H, int32_t Hkv, int32_t groups, int32_t* boxes, int32_t max_boxes) {
  if (B < 1 || H < 1) return 0;
  if (Hkv <= 0) Hkv = H;
  if (Hkv > H || H % Hkv != 0 || groups < 1) return 0;
  const std::vector<Box> v = head_groups(B, H, Hkv, groups);
  for (size_t i = 0; boxes && i < v.size() && (int32_t)i < max_boxes; ++i) {
    boxes[4 * i] = v[i].b0; boxes[4 * i + 1] = v[i].b1; boxes[4 * i + 2] = v[i].h0; boxes[4 * i + 3] = v[i].h1;
  }
  return (int32_t)v.size();
}

size_t sparsepr_call_host_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                          int32_t groups) {
  std::vector<Box> boxes;
  Layout L;
  return lay_out(shape, params, groups, &boxes, &L) ? L.total : 0;
}

sparsepr_status_t sparsepr_call_host(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                     const void* Q_host, const void* K_host, const void* V_host, void* O_host,
                                     int32_t groups, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!Q_host || !K_host || !V_host || !O_host) return SPARSEPR_ERR_INVALID_ARG;
  std::vector<Box> boxes;
  Layout L;
  if (!lay_out(shape, params, groups, &boxes, &L)) return SPARSEPR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < L.total) return SPARSEPR_ERR_WORKSPACE;
  Pipe* pipe = acquire_pipe();
  const size_t ng = boxes.size();
  if (!pipe || !pipe->grow(3 * ng + 3)) { release_pipe(pipe); return SPARSEPR_ERR_CUDA; }
  cudaStream_t s_main = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const int Hkv = shape->Hkv > 0 ? shape->Hkv : shape->H, G = shape->H / Hkv;
  const size_t nd = (size_t)shape->N * shape->d * L.es;          // bytes of one head
  cudaEvent_t* ev = pipe->ev.data();
  cudaEvent_t ev_start = ev[3 * ng], ev_work = ev[3 * ng + 1], ev_down = ev[3 * ng + 2];
  bool ok = true;
  auto chk = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };
  // earlier work on `cuda_stream` (which may still use the workspace) comes first
  chk(cudaEventRecord(ev_start, s_main));
  chk(cudaStreamWaitEvent(pipe->up, ev_start, 0));
  chk(cudaStreamWaitEvent(pipe->work, ev_start, 0));
  chk(cudaStreamWaitEvent(pipe->down, ev_start, 0));
  // uploads: Q and K of a group (all the plan needs), then its V
  for (size_t g = 0; ok && g < ng; ++g) {
    const Box& b = boxes[g];
    const size_t qoff = ((size_t)b.b0 * shape->H + b.h0) * nd, koff = ((size_t)b.b0 * Hkv + b.h0 / G) * nd;
    const size_t qn = ((size_t)(b.b1 - b.b0 - 1) * shape->H + (b.h1 - b.h0)) * nd;
    const size_t kn = ((size_t)(b.b1 - b.b0 - 1) * Hkv + (b.h1 - b.h0) / G) * nd;
    chk(cudaMemcpyAsync(ws + L.q + qoff, static_cast<const char*>(Q_host) + qoff, qn, cudaMemcpyHostToDevice, pipe->up));
    chk(cudaMemcpyAsync(ws + L.k + koff, static_cast<const char*>(K_host) + koff, kn, cudaMemcpyHostToDevice, pipe->up));
    chk(cudaEventRecord(ev[3 * g], pipe->up));
    chk(cudaMemcpyAsync(ws + L.v + koff, static_cast<const char*>(V_host) + koff, kn, cudaMemcpyHostToDevice, pipe->up));
    chk(cudaEventRecord(ev[3 * g + 1], pipe->up));
  }
  std::vector<sparsepr_plan_t*> plans(ng, nullptr);
  sparsepr_status_t st = ok ? SPARSEPR_OK : SPARSEPR_ERR_CUDA;
  for (size_t g = 0; st == SPARSEPR_OK && g < ng; ++g) {
    const Box& b = boxes[g];
    cudaStream_t w = (g & 1) ? pipe->work : s_main;
    const sparsepr_shape_t t = sub_shape(*shape, Hkv, b);
    sparsepr_params_t p = *params;
    p.head_offset = params->head_offset + b.b0 * shape->H + b.h0;
    const size_t qoff = ((size_t)b.b0 * shape->H + b.h0) * nd, koff = ((size_t)b.b0 * Hkv + b.h0 / G) * nd;
    const size_t qn = ((size_t)(b.b1 - b.b0 - 1) * shape->H + (b.h1 - b.h0)) * nd;
    chk(cudaStreamWaitEvent(w, ev[3 * g], 0));
    if (!ok) { st = SPARSEPR_ERR_CUDA; break; }
    st = sparsepr_plan(&t, &p, ws + L.q + qoff, ws + L.k + koff, ws + L.v + koff, ws + L.plan_off[g], L.plan_bytes[g], w,
                       &plans[g]);
    if (st != SPARSEPR_OK) break;
    chk(cudaStreamWaitEvent(w, ev[3 * g + 1], 0));
    if (!ok) { st = SPARSEPR_ERR_CUDA; break; }
    st = sparsepr_attend(plans[g], ws + L.q + qoff, ws + L.k + koff, ws + L.v + koff, ws + L.o + qoff, nullptr,
                         ws + L.att_off[g], L.att_bytes[g], w);
    if (st != SPARSEPR_OK) break;
    chk(cudaEventRecord(ev[3 * g + 2], w));
    chk(cudaStreamWaitEvent(pipe->down, ev[3 * g + 2], 0));
    chk(cudaMemcpyAsync(static_cast<char*>(O_host) + qoff, ws + L.o + qoff, qn, cudaMemcpyDeviceToHost, pipe->down));
    if (!ok) st = SPARSEPR_ERR_CUDA;
  }
  // join: everything queued above is complete before the call returns, whatever happened
  cudaEventRecord(ev_work, pipe->work);
  cudaStreamWaitEvent(s_main, ev_work, 0);
  cudaEventRecord(ev_down, pipe->down);
  cudaStreamWaitEvent(s_main, ev_down, 0);
  const cudaError_t e_up = cudaStreamSynchronize(pipe->up), e_main = cudaStreamSynchronize(s_main);
  if (st == SPARSEPR_OK && (e_up != cudaSuccess || e_main != cudaSuccess)) st = SPARSEPR_ERR_CUDA;
  if (st == SPARSEPR_OK) {
    // a device-side error word (bounded wait that ran out, invalid intermediate) of any group fails the call
    for (size_t g = 0; g < ng && st == SPARSEPR_OK; ++g) {
      int32_t word = 0;
      const sparsepr_status_t s2 = sparsepr_plan_device_error(plans[g], &word);
      if (s2 != SPARSEPR_OK) st = s2;
      else if (word != 0) st = static_cast<sparsepr_status_t>(word);
    }
  }
  for (sparsepr_plan_t* pl : plans)
    if (pl) sparsepr_plan_destroy(pl);
  release_pipe(pipe);
  return st;
}

}  // extern "C"
