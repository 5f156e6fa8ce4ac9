/*
 * sparsepr.h -- C ABI of the SparsePR attention library for NVIDIA B200 (sm_100a).
 *
 * One call replaces dense self-attention O = softmax(s Q K^T) V (Eq. 1 of the
 * SparsePR paper) for every (batch, head) of a long token sequence by
 *   plan   : Response-Coupled Partitioning (Section 4.1, Appendix B), group-major
 *            permutations, probe selection (Algorithm A.1) and routing under a
 *            query-key pair budget (Section 4.3);
 *   attend : block-sparse attention with renormalised hard drop (Eq. 3), exact
 *            probe rows, the weighted ridge fit restricted to the probe-residual
 *            subspace (Eq. 8-9, Appendix A.3) and the corrected output (Eq. 10),
 *            written back in the original token order.
 *
 * Conventions
 *   - Every pointer argument is marked HOST or DEVICE.  Device pointers must be
 *     valid on the CUDA device that is current when the call is made.
 *   - Q, K, V, O are [B, H, N, d] tensors addressed through element strides for
 *     B, H and N; the last dimension is contiguous.  Rows must start on a
 *     16-byte boundary.  N_q = N_k = N and d_v = d.  K and V may have fewer heads
 *     than Q (grouped-query attention, sparsepr_shape_t.Hkv).
 *   - The library never allocates or frees device memory: the caller owns all
 *     tensors and both workspaces.  A plan handle is a small host object that
 *     points into the plan workspace; it is valid until the workspace is released
 *     or sparsepr_plan_destroy is called.  Process-wide state is limited to what is
 *     set up once and then reused: kernel attributes and the tensor-map encoder
 *     (first call), a pool of auxiliary streams and events (two streams and three
 *     events per plan alive at the same time, per device; created when the pool is
 *     empty, returned by sparsepr_plan_destroy, never freed), the SM count per
 *     device, and the scratch array of sparsepr_stage_assign_static.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*)
 *     and is asynchronous, except the calls documented as synchronising.
 *   - Errors are return codes.  Argument errors are detected before anything
 *     is launched.  Conditions found on the device (non-finite input, a
 *     breakdown of the Cholesky factorisation, a bounded wait that ran out)
 *     are recorded in a device error word that sparsepr_plan_stats reports.
 *     The word lives in the plan workspace and persists for the life of the plan;
 *     once a bounded wait has run out (SPARSEPR_ERR_TIMEOUT) the tensor-core
 *     kernels of later calls on that plan return at once, so O is undefined
 *     whenever `device_error` is non-zero.  No call aborts, throws or traps.
 */
#ifndef SPARSEPR_H_
#define SPARSEPR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPARSEPR_OK = 0,
  SPARSEPR_ERR_INVALID_ARG = 1,
  SPARSEPR_ERR_UNSUPPORTED = 2,
  SPARSEPR_ERR_WORKSPACE = 3,   /* workspace too small or misaligned (256 B) */
  SPARSEPR_ERR_CUDA = 4,
  SPARSEPR_ERR_NUMERIC = 5,
  SPARSEPR_ERR_TIMEOUT = 6
} sparsepr_status_t;

typedef enum { SPARSEPR_F32 = 0, SPARSEPR_BF16 = 1 } sparsepr_dtype_t;

/* How the two partitions are built: the method, and the two ablation variants of Section 5.2 (Table 2).  The
 * semantic reference partition of Section 3.1 applies k-means to the key and to the query activations
 * themselves; the key-response K/V variant changes only the K/V partition.  Initial rows, iteration count and
 * tie rules are the same in every variant.  Where the query partition is semantic, Algorithm A.1 ranks the probe
 * candidates by their distance in the raw query space.  The variants cluster in d dimensions on the CUDA cores
 * (d = 128: several times the cost of the method's 64-dimensional tensor-core k-means). */
typedef enum {
  SPARSEPR_PARTITION_RESPONSE_COUPLED = 0,
  SPARSEPR_PARTITION_KEY_RESPONSE_KV = 1,
  SPARSEPR_PARTITION_SEMANTIC = 2
} sparsepr_partition_t;

/* Problem shape: Q, K in R^{N x d}, V in R^{N x d_v} per (batch, head) -- the
 * paper's problem statement (Section 3).  Strides are in elements. */
typedef struct {
  int32_t B, H, N, d, dv;
  int32_t dtype;                       /* sparsepr_dtype_t of Q, K, V and O */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];   /* B, H, N */
  /* Grouped-query attention: number of K/V heads (0 or H = ordinary multi-head attention; must divide H).  K and V
   * are then [B, Hkv, N, d] (their head strides count K/V heads) and query head h attends to K/V head
   * h / (H / Hkv).  The K/V partition, permutation, offsets and centroids are computed once per K/V head from the
   * pooled query samples of its query heads and shared by them (Section 4.3); every query head keeps its own query
   * partition, probes and routes.  Per-K/V-head arrays of sparsepr_plan_host_t and sparsepr_plan_features_t
   * (kv_assign, kv_perm, kv_off, F_K, F_Q, kappa) have B*Hkv entries.  bf16, d = 128 only. */
  int32_t Hkv;
} sparsepr_shape_t;

/* Method parameters (Appendix C, Table C.1, plus the knobs the paper leaves
 * open).  A zero in a field with a stated default selects the default. */
typedef struct {
  float density;         /* target rho_exec, probes included (Section 4.3); >= 1 selects every cell */
  int32_t block;         /* nominal group size: C_k = C_q = ceil(N / block) unless given below */
  int32_t Ck, Cq;        /* number of K/V groups and of query groups; 0 = derive from block */
  int32_t n_sample;      /* M_s sampled query rows for the key-response metric (Appendix B.1) */
  int32_t n_probe;       /* M exact probe rows per head (Appendix A.2) */
  int32_t rK, rQ;        /* feature ranks, defaults 48 and 64, clamped to d */
  int32_t r_out;         /* probe-residual output rank r, default 16, clamped to min(M, d_v) */
  float lambda;          /* ridge coefficient (Eq. 8); negative selects the default 0.1, 0 is honoured */
  float eps_rms;         /* stabiliser of the RMS normalisation (Eq. 7), default 1e-6 */
  float eps_std;         /* epsilon inside the feature scale s_x (Appendix A.3), default 1e-6 */
  int32_t kmeans_iters;  /* Lloyd iterations T (assignments), default 8 */
  float softmax_scale;   /* s; 0 selects 1/sqrt(d) */
  uint64_t seed;         /* offsets the deterministic row samples */
  int32_t mode;          /* 0 = probe-fitted reconstruction, 1 = renormalised hard drop only */
  int32_t partition;     /* sparsepr_partition_t; 0 = Response-Coupled Partitioning */
  int32_t head_offset;   /* The deterministic row samples (Appendix B.1: sampled queries; k-means initialisation) are keyed by
                          * head_offset + b H + h.  A problem cut into groups of heads, each group a call of its own with the
                          * index of its first head here, gives bit for bit the plan of one call over all heads (outputs agree up to
                          * the summation order of the probe rows, whose key slices are sized per call).
                          * >= 0 and a multiple of H / Hkv; 0 for a whole problem. */
} sparsepr_params_t;

typedef struct sparsepr_plan_s sparsepr_plan_t;

/* Densities and group statistics of a plan, aggregated over all heads
 * (Eq. 2 and Section 4.3).  `device_error` is 0 or the sparsepr_status_t that
 * a kernel recorded. */
typedef struct {
  int64_t routed_pairs;        /* sum over heads of sum_ab z_ab |G_a||G_b| */
  int64_t routed_cells;        /* number of selected cells */
  int64_t padded_tile_pairs;   /* pairs the block-sparse kernel issues, padding included */
  double rho_route, rho_exec;  /* mean over heads */
  double rho_route_min, rho_route_max;
  int32_t nonempty_kv_groups_min, nonempty_q_groups_min;
  int32_t max_kv_group, max_q_group;
  int32_t assign_rechecked_rows;   /* rows of the last k-means assignments decided by the exact recheck */
  int32_t device_error;
  /* Lloyd passes that ran on the K/V side and on the query side (largest count over heads).  A head stops
   * early when a pass changes no assignment: every later pass would repeat it exactly, so the result is
   * the one of all T passes.  0 for an imported plan. */
  int32_t kmeans_passes_kv, kmeans_passes_q;
} sparsepr_stats_t;

/* Host-side view of a plan, one entry per (batch, head) in b-major order, used
 * to export a plan for inspection and to import one made elsewhere.  Every
 * pointer is HOST memory owned by the caller; NULL skips the field on export.
 *   kv_assign, q_assign : [BH, N]   group id of every token (Section 3)
 *   kv_perm, q_perm     : [BH, N]   original index of the token at each group-major position
 *   kv_off, q_off       : [BH, C+1] ragged group offsets
 *   route_ptr           : [BH, Cq+1]; route_idx : [BH, Cq*Ck] slab per head, rows ascending in b
 *   probe_idx, probe_w  : [BH, M]   probe rows in selection order and coverage weights w_p
 *   routed_pairs        : [BH]
 */
typedef struct {
  int32_t *kv_assign, *q_assign;
  int32_t *kv_perm, *q_perm;
  int32_t *kv_off, *q_off;
  int32_t *route_ptr, *route_idx;
  int32_t *probe_idx;
  float *probe_w;
  int64_t *routed_pairs;
} sparsepr_plan_host_t;

/* Floating-point intermediates of a plan (Section 4.1, Appendix B; the router's group means and cell
 * scores of Section 4.3), exported so that they can be compared with an independent evaluation.  Every
 * pointer is HOST memory owned by the caller; NULL skips the field.  All float32, b-major over (batch, head):
 *   F_K   [BH, d, r_K], F_Q [BH, d, r_Q]  feature maps (columns = scaled eigendirections; their signs are arbitrary)
 *   phi_Q [BH, N, r_Q]                    RMS-normalised query responses (Eq. 7); [BH, N, d] raw queries when the
 *                                         query partition is semantic (F_Q, and F_K for the semantic K/V partition,
 *                                         are then not written)
 *   kappa [BH, C_k, d], theta [BH, C_q, d] original-space means of the K/V groups and of the query groups
 *   score [BH, C_q, C_k]                  cell scores the router selected from */
typedef struct {
  float *F_K, *F_Q, *phi_Q, *kappa, *theta, *score;
} sparsepr_plan_features_t;

/* Stages of one call, in launch order, as indices into sparsepr_profile_t.ms.  Plan
 * (Section 4.1, 4.3, Algorithm A.1): KEY_METRIC = sampled-query Gram and its
 * eigen-decomposition; *_PROJECT = response coordinates (Eq. 6, Eq. 7); *_KMEANS;
 * *_PERMUTE = counting sort and group means; QUERY_METRIC = centroid Gram and its
 * eigen-decomposition; PROBE_SELECT; ROUTE = cell scores and selection.  Attend:
 * GATHER = group-major copies of Q, K, V; PROBE_ROWS = exact and hard-drop rows of
 * the probes; FIT = ridge fit and subspace; ATTENTION = block-sparse kernels (the 128-row
 * tiles and the packed group remainders, side by side on two streams);
 * CORRECTION = residual correction of Eq. 9 (zero where the block-sparse kernel applies
 * it in its epilogue); PROBE_WRITE.  DENSE = the dense entry point.  A call without a
 * profile runs PROBE_SELECT beside ROUTE and PROBE_ROWS + FIT beside ATTENTION on a second
 * stream, so its duration is less than the sum of the stages. */
enum {
  SPARSEPR_STAGE_KEY_METRIC = 0, SPARSEPR_STAGE_KEY_PROJECT, SPARSEPR_STAGE_KEY_KMEANS, SPARSEPR_STAGE_KEY_PERMUTE,
  SPARSEPR_STAGE_QUERY_METRIC, SPARSEPR_STAGE_QUERY_PROJECT, SPARSEPR_STAGE_QUERY_KMEANS, SPARSEPR_STAGE_QUERY_PERMUTE,
  SPARSEPR_STAGE_PROBE_SELECT, SPARSEPR_STAGE_ROUTE,
  SPARSEPR_STAGE_GATHER, SPARSEPR_STAGE_PROBE_ROWS, SPARSEPR_STAGE_FIT, SPARSEPR_STAGE_ATTENTION,
  SPARSEPR_STAGE_CORRECTION, SPARSEPR_STAGE_PROBE_WRITE, SPARSEPR_STAGE_DENSE, SPARSEPR_STAGE_COUNT
};
/* Milliseconds per stage, measured with CUDA events on the call's stream.  The
 * *_timed calls ADD to the entries, so one zero-initialised struct can accumulate
 * several calls. */
typedef struct { float ms[SPARSEPR_STAGE_COUNT]; } sparsepr_profile_t;

const char* sparsepr_status_string(sparsepr_status_t s);

/* Bytes of DEVICE workspace that sparsepr_plan / sparsepr_plan_import and
 * sparsepr_attend need for this shape and these parameters.  0 on invalid input. */
size_t sparsepr_plan_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params);
size_t sparsepr_attend_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params);

/* Stages 1-2 (Sections 4.1 and 4.3, Algorithm A.1): builds partition, permutations,
 * probe set and routes of every head from Q and K (DEVICE, read only; V is not
 * read -- values never enter the partition features -- and may be NULL).
 * `workspace` is DEVICE memory of at least sparsepr_plan_workspace_bytes, 256-byte
 * aligned; the plan lives in it.  *out receives a HOST handle.  The probe selection may
 * still be running on a stream of the plan's own when the call returns: sparsepr_attend
 * orders its work behind it, sparsepr_plan_stats / _export / _destroy wait for it, so the
 * workspace may be released once sparsepr_plan_destroy has returned and the work queued on
 * `cuda_stream` is complete. */
sparsepr_status_t sparsepr_plan(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                const void* Q, const void* K, const void* V,
                                void* workspace, size_t workspace_bytes, void* cuda_stream,
                                sparsepr_plan_t** out);

/* The same with warm-started k-means (Appendix C.1: "warm-started GPU k-means"), for a sequence of calls over
 * the same token grid, e.g. successive denoising steps.  prev_kv_assign, prev_q_assign: DEVICE int32 [B*H, N], the
 * partition of an earlier call (group ids in [0, C_k) and [0, C_q); other values are ignored).  The initial centroid
 * of a group is the mean of the CURRENT features of the tokens that partition put into it; a group it left empty
 * starts from its strided sample row as in sparsepr_plan.  Seeding by assignment rather than by centroids makes the
 * start independent of the sign gauge of the eigenvectors behind the feature maps, which can change between calls.
 * params->kmeans_iters still counts the assignment passes, and fewer are needed (the benchmark's warm leg uses 2).
 * The arrays may live in an earlier plan's workspace (see sparsepr_plan_assignments); they are read by work queued
 * on `cuda_stream` and must stay valid until that work is complete. */
sparsepr_status_t sparsepr_plan_warm(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                     const void* Q, const void* K, const void* V,
                                     const int32_t* prev_kv_assign, const int32_t* prev_q_assign,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream,
                                     sparsepr_plan_t** out);

/* DEVICE pointers to the partition inside the plan's workspace: int32 [B*H, N] each, valid while the workspace
 * lives; their contents are final once the work of the plan call is complete on its stream. */
sparsepr_status_t sparsepr_plan_assignments(const sparsepr_plan_t* plan, const int32_t** kv_assign,
                                            const int32_t** q_assign);

/* Stages 3-4 (Eq. 3, Eq. 8-10): O (DEVICE, written in original token order) from
 * Q, K, V (DEVICE) and a plan.  `workspace`: DEVICE, sparsepr_attend_workspace_bytes,
 * 256-byte aligned; its contents are scratch.  `O_sparse` (DEVICE, float32
 * [B,H,N,dv] contiguous, may be NULL) additionally receives the uncorrected
 * hard-drop output O^sp in original order, for error reporting. */
sparsepr_status_t sparsepr_attend(const sparsepr_plan_t* plan, const void* Q, const void* K, const void* V,
                                  void* O, float* O_sparse, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);

/* Dense attention, Eq. 1, with the same kernels run over the full key range.
 * Needs no workspace.  softmax_scale 0 selects 1/sqrt(d). */
sparsepr_status_t sparsepr_dense(const sparsepr_shape_t* shape, float softmax_scale,
                                 const void* Q, const void* K, const void* V, void* O, void* cuda_stream);

/* A whole call for tensors in HOST memory (Stages 1-4 plus the copies): Q, O contiguous [B, H, N, d], K, V
 * contiguous [B, Hkv, N, d] in (preferably pinned) host memory; the stride fields of `shape` are ignored.  Heads are
 * independent (Section 4.3 shares only the K/V partition inside a group of query heads), so the problem is cut into
 * `groups` groups of consecutive heads (sparsepr_head_groups) that move through a pipeline: one stream uploads group
 * after group, two streams take the groups in turn through sparsepr_plan + sparsepr_attend, a fourth returns every
 * group's O.  A group runs with head_offset = params->head_offset + its first head, so its plan is that of one call
 * over all heads.  `workspace`: DEVICE, sparsepr_call_host_workspace_bytes(shape, params, groups), 256-byte aligned;
 * it receives the device copies of Q, K, V, O and the workspaces of every group.  The call returns when O is
 * complete in host memory (it synchronises `cuda_stream` and its own streams).  groups < 1 selects 4. */
size_t sparsepr_call_host_workspace_bytes(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                          int32_t groups);
sparsepr_status_t sparsepr_call_host(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                     const void* Q_host, const void* K_host, const void* V_host, void* O_host,
                                     int32_t groups, void* workspace, size_t workspace_bytes, void* cuda_stream);
/* The groups of that pipeline: boxes[4 i .. 4 i + 3] = {b0, b1, h0, h1}, heads [h0, h1) of the batch entries
 * [b0, b1); either one batch entry with a range of heads (a multiple of H / Hkv at both ends) or whole batch
 * entries, in the order b H + h.  Writes at most max_boxes boxes and returns the number of groups (at most
 * groups + B), 0 on invalid arguments.  HOST only, no GPU needed. */
int32_t sparsepr_head_groups(int32_t B, int32_t H, int32_t Hkv, int32_t groups, int32_t* boxes, int32_t max_boxes);

/* The same calls with per-stage timing (the latency decomposition of the paper's
 * Section 5.3): identical work and results; they record CUDA events between the
 * stages, synchronise the stream before returning and add the elapsed
 * milliseconds to *profile (HOST). */
sparsepr_status_t sparsepr_plan_timed(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                      const void* Q, const void* K, const void* V,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream,
                                      sparsepr_plan_t** out, sparsepr_profile_t* profile);
sparsepr_status_t sparsepr_attend_timed(const sparsepr_plan_t* plan, const void* Q, const void* K, const void* V,
                                        void* O, float* O_sparse, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream, sparsepr_profile_t* profile);
sparsepr_status_t sparsepr_dense_timed(const sparsepr_shape_t* shape, float softmax_scale,
                                       const void* Q, const void* K, const void* V, void* O, void* cuda_stream,
                                       sparsepr_profile_t* profile);

/* Synchronises the stream the plan was built on, then fills *host_out. */
sparsepr_status_t sparsepr_plan_stats(const sparsepr_plan_t* plan, sparsepr_stats_t* host_out);
/* Only the device error word of the plan and of the attend calls made with it so far (what sparsepr_plan_stats
 * reports as `device_error`): waits for the plan's streams and copies one word. */
sparsepr_status_t sparsepr_plan_device_error(const sparsepr_plan_t* plan, int32_t* device_error);
sparsepr_status_t sparsepr_plan_export(const sparsepr_plan_t* plan, sparsepr_plan_host_t* host_out);

/* Synchronises like sparsepr_plan_export, then copies the requested intermediates.  A plan made by
 * sparsepr_plan_import has none: SPARSEPR_ERR_UNSUPPORTED. */
sparsepr_status_t sparsepr_plan_export_features(const sparsepr_plan_t* plan, sparsepr_plan_features_t* host_out);

/* Builds a plan from host-side assignments, routes (CSR slabs as in
 * sparsepr_plan_host_t) and probes; permutations and offsets are recomputed on
 * the device.  Used to run stages 3-4 on a partition produced elsewhere. */
sparsepr_status_t sparsepr_plan_import(const sparsepr_shape_t* shape, const sparsepr_params_t* params,
                                       const sparsepr_plan_host_t* host_in,
                                       void* workspace, size_t workspace_bytes, void* cuda_stream,
                                       sparsepr_plan_t** out);

/* Frees the HOST handle only. */
void sparsepr_plan_destroy(sparsepr_plan_t* plan);

/* ---- single stages, exposed so that the integer work can be checked bit for bit ---- */

/* a[j] = argmin_c sum_k (X[j,k]-mu[c,k])^2 with ties to the lowest c: the
 * assignment step of k-means (Section 4.1).  X [n,r], mu [C,r] float32 DEVICE,
 * a [n] int32 DEVICE.  The decision equals the one taken in float64 with the
 * terms accumulated in order of k.  `ws`: DEVICE scratch of at least
 * sparsepr_stage_assign_workspace_bytes(n, C, r). */
size_t sparsepr_stage_assign_workspace_bytes(int32_t n, int32_t C, int32_t r);
sparsepr_status_t sparsepr_stage_assign(int32_t n, int32_t C, int32_t r, const float* X, const float* mu,
                                        int32_t* a, void* ws, size_t ws_bytes, void* cuda_stream);

/* The assignment stage for callers that cannot allocate.  The paper has no
 * counterpart of this call; it exists for users of the library such as a plug-in
 * that runs inside an inference server which has already handed every byte of
 * device memory to its own pool, or a control loop that may not call cudaMalloc
 * because of the device-wide synchronisation an allocation implies.  Such a caller
 * has nowhere to get the workspace of sparsepr_stage_assign from.  Here the scratch
 * is a fixed array inside the library image (about 4.3 MB on every GPU that loads
 * the library, held until the process exits), so only the inputs X [n,r], mu [C,r]
 * (float32, DEVICE) and the output a [n] (int32, DEVICE) are passed.  The result is
 * identical to sparsepr_stage_assign.
 *   - Limits: n <= 16384, C <= 1024, r <= 64.  Anything larger is refused with
 *     SPARSEPR_ERR_UNSUPPORTED ("unsupported shape or parameter") before any launch.
 *   - The call allocates and frees nothing, on the device or through any library.
 *   - The first call on each device looks up the device address of the array (with
 *     that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array, which still holds the previous
 *     call's data; every element that is read is rewritten first, so nothing has
 *     to be cleared by the caller.  Two calls that may run on the GPU at the same
 *     time (different streams, different threads) race on it: serialise them. */
sparsepr_status_t sparsepr_stage_assign_static(int32_t n, int32_t C, int32_t r, const float* X, const float* mu,
                                               int32_t* a, void* cuda_stream);

/* Stable counting sort by group id (Section 4.3, group-major layout):
 * perm [n], inv [n], off [C+1], all int32 DEVICE. */
sparsepr_status_t sparsepr_stage_permute(int32_t n, int32_t C, const int32_t* a,
                                         int32_t* perm, int32_t* inv, int32_t* off, void* cuda_stream);

/* Cell selection under a pair budget (Section 4.3) for one head from given
 * float32 cell scores [Cq,Ck], group sizes nq [Cq], nk [Ck] (int32) -- all DEVICE.
 * Writes route_ptr [Cq+1], route_idx [Cq*Ck] (ascending inside a row) and
 * *pairs_out (int64), all DEVICE.  select_all != 0 takes every non-empty cell. */
sparsepr_status_t sparsepr_stage_route(int32_t Cq, int32_t Ck, const float* score,
                                       const int32_t* nq, const int32_t* nk, int64_t pair_budget,
                                       int32_t select_all, int32_t* route_ptr, int32_t* route_idx,
                                       int64_t* pairs_out, void* cuda_stream);

/* Self-test of the bounded device waits.  Every wait of a tensor-core kernel on an mbarrier gives up after a
 * cycle limit, records SPARSEPR_ERR_TIMEOUT and lets the kernel return, so that a lost copy cannot hang the
 * device.  This call runs that wait into its limit on purpose in the harmless form: one warp waits, for 2^16
 * cycles (tens of microseconds), on a barrier that nothing arrives at -- no copy is in flight and no tensor memory
 * is held.  Afterwards *device_error_word (DEVICE int32, zeroed by the caller) holds SPARSEPR_ERR_TIMEOUT, and
 * the context is as usable as before. */
sparsepr_status_t sparsepr_selftest_bounded_wait(int32_t* device_error_word, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* SPARSEPR_H_ */
