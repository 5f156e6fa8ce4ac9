// Internal launch interface between the C-ABI layer and the kernels.
#pragma once
#include "common.cuh"

namespace spr {

// Number of SMs of the current device (cached per device; 148 when no device can be queried, so that
// workspace sizes can still be computed).  Defined in api.cu.
int sm_count();

// ---- partition.cu -------------------------------------------------------------
cudaError_t init_group_sort();
void launch_sample_gram(int dtype, const void* Q, const i64* qs, int BH, int H, int N, int d, int Ms, u64 seed, int head0,
                        double* Mout, cudaStream_t st);
void launch_centroid_gram(const float* kappa, const int* n, int BH, int C, int d, double* Mout, cudaStream_t st);
// eigen.cu: leading r <= 64 eigenpairs of `batch` symmetric n x n matrices (n = 64 or 128), `stride` doubles apart.
// scale_mode 0: columns scaled by sqrt(lambda_j / mean retained lambda); 1: orthonormal columns; precise: float64.
// Fout [batch][n][r]; lam_out [batch][n] or null; ws: eig_scratch_doubles(batch, n) doubles of scratch.
cudaError_t init_eigen();
size_t eig_scratch_doubles(int batch, int n);
void launch_eig_top(const double* Min, i64 stride, int batch, int n, int r, int scale_mode, bool precise, float* Fout,
                    double* lam_out, double* ws, cudaStream_t st);
void launch_project(int dtype, const void* X, const i64* xs, int BH, int H, int N, int d, int r, const float* F,
                    bool rms, float eps, float* phi, int ldphi, unsigned* maxabs, int* err, cudaStream_t st);
// features of the semantic partition: the activations themselves as float32 rows [BH][N][d]
void launch_raw_features(int dtype, const void* X, const i64* xs, int BH, int H, int N, int d, float* phi, unsigned* maxabs,
                         int* err, cudaStream_t st);
void launch_kmeans_init(const float* phi, int ldphi, int BH, int N, int r, int C, u64 seed, int tag, int head0, float* mu,
                        i64* sums, int* counts, const unsigned* maxabs_bits, int* fx_shift, cudaStream_t st);
void launch_kmeans_warm_sums(const float* phi, int ldphi, int BH, int N, int r, int C, const int* prev, i64* sums,
                             int* counts, const int* fx_shift, cudaStream_t st);
void launch_kmeans_finalize(float* mu, float* mu2, float* mumax, i64* sums, int* counts, const int* fx_shift, int BH,
                            int C, int r, int update, cudaStream_t st, __nv_bfloat16* mh = nullptr, __nv_bfloat16* ml = nullptr);
// prev_changed / cur_changed [BH] (may be null): number of rows of each head whose assignment changed in the previous
// / this pass.  A head whose previous pass changed nothing is skipped (Lloyd's iteration has reached its fixed
// point: every later pass would reproduce the same assignment and the same centroids).
void launch_kmeans_assign(const float* phi, int ldphi, int BH, int N, int r, const float* mu, const float* mu2,
                          const float* mumax, int C, int* assign, i64* sums, int* counts, const int* fx_shift,
                          int* recheck_count, const int* prev_changed, int* cur_changed, cudaStream_t st);
void launch_group_sort(const int* assign, int BH, int N, int C, int* perm, int* inv, int* off, int* err, cudaStream_t st);
void launch_group_means(int dtype, const void* X, const i64* xs, int BH, int H, const int* perm, const int* off, int N,
                        int C, int d, float* out, int* sizes, cudaStream_t st);
void launch_gather_rows(int dtype, const void* X, const i64* xs, int BH, int H, const int* perm, int N, int d, void* out,
                        cudaStream_t st);

// project_tc.cu: the same projection on the tensor cores (bf16, d = 128, r <= 64); Ft: bf16 scratch [BH][3][64][128]
cudaError_t init_project_tc();
bool project_tc_supported(int dtype, int d, int r, const i64* xs);
// f_div: heads that share one feature map (F is indexed by bh / f_div)
bool launch_project_tc(const void* X, const i64* xs, int BH, int H, int N, int r, const float* F, bool rms, float eps,
                       float* phi, int ldphi, unsigned* maxabs, __nv_bfloat16* Ft, int* err, cudaStream_t st, int f_div = 1);

// ---- kmeans_tc.cu (tcgen05 score contraction + exact recheck) --------------------------------------
struct KmeansTcArgs {
  int BH, N, C, r, R;
  const __nv_bfloat16 *xh, *xl, *mh, *ml;      // [BH][N][64], [BH][C][64] split operands
  const float* phi; int ldphi;                 // fp32 features [BH][N][ldphi]
  const float *xnorm, *mu, *mu2;               // [BH][N], [BH][C][R], [BH][C]
  int* assign;
  i64* sums; int* counts; const int* fx_shift; // null sums = assignment only
  int *flagged, *flag_count, *recheck_total, *err;   // flagged [BH][N] scratch, flag_count [BH] scratch, recheck_total: rows rechecked by this pass
  const int* prev_changed; int* cur_changed;   // [BH] or null, as for launch_kmeans_assign
  int* flag_count_next;                        // [BH] or null: the next pass's counters, zeroed by this pass (flag_count itself must arrive zeroed)
};
cudaError_t init_kmeans_tc();
bool kmeans_tc_supported();
void launch_split_bf16(const float* x, int ld, i64 rows, int r, __nv_bfloat16* hi, __nv_bfloat16* lo, float* norm,
                       cudaStream_t st);
bool launch_kmeans_assign_tc(const KmeansTcArgs& a, cudaStream_t st);

// ---- routing.cu ---------------------------------------------------------------
struct RouteState {      // per head, device
  i64 pairs;             // routed pairs
  i64 cells;             // selected cells
};
// kv_div = query heads per K/V head: kappa and nk (K/V side) are indexed by bh / kv_div
void launch_cell_scores(const float* theta, const float* kappa, const int* nq, const int* nk, int BH, int Cq, int Ck,
                        int d, float scale, float* score, int kv_div, cudaStream_t st);
void launch_route_select(const float* score, const int* nq, const int* nk, int BH, int Cq, int Ck, i64 budget,
                         int select_all, int* route_ptr, int* route_idx, RouteState* state, i64* pairs_out,
                         int kv_div, cudaStream_t st);
void launch_count_pairs(const int* q_off, const int* kv_off, const int* route_ptr, const int* route_idx, int BH, int Cq,
                        int Ck, RouteState* state, int kv_div, cudaStream_t st);
cudaError_t init_routing();
void launch_probe_select(const float* phiQ, int ldphi, int r, const int* q_perm, const int* q_off, const int* nq, int BH,
                         int N, int Cq, int M, double* dist_scratch, int* probe_idx, float* probe_w, cudaStream_t st);

// ---- attention_simt.cu ----------------------------------------------------------
struct AttnArgs {
  int dtype, BH, H, N, d;
  float scale;
  // group-major inputs [BH][N][d] (sparse) or strided originals (dense)
  const void *Q, *K, *V;
  i64 qs[3], ks[3], vs[3];
  // sparse metadata (null for dense)
  const int *q_off, *kv_off, *route_ptr, *route_idx, *q_perm, *tile_off;
  int Cq, Ck;
  int kv_div;                 // query heads per K/V head (grouped-query attention): K/V-side arrays are indexed by bh / kv_div; 0 = 1
  // epilogue
  const float *A, *c;         // [BH][d][d], [BH][d]; null = no correction
  void* O; i64 os[3];
  float* O_sparse;            // optional [BH][N][d] in original order
  void* O_lo;                 // optional bf16 [BH][N][d] in original order: o - bf16(o) (tensor-core kernels only)
  int* err;                   // device error word (may be null)
};
cudaError_t init_attention_simt();
// tile_off [BH][Cq+1]: prefix of the tiles per query group; small_rem > 0 leaves out a last tile of at most small_rem rows
void launch_tile_offsets(const int* q_off, int BH, int Cq, int tile_rows, int small_rem, int* tile_off, cudaStream_t st);
void launch_attention_simt(const AttnArgs& a, cudaStream_t st);
// ---- attention_tc.cu (tcgen05 / TMEM / TMA; bf16, d = 128) -------------------------------------
cudaError_t init_attention_tc();
bool attention_tc_supported(const AttnArgs& a);
// tile_off in `a` must have been built for 128-row tiles; a.A and a.c are ignored (no correction epilogue)
bool launch_attention_tc(const AttnArgs& a, cudaStream_t st);
// Query-group remainders of 1..kRemRows rows are left out of the 128-row kernel's tiles (tile offsets built with
// small_rem = kRemRows) and handled by attention_packed.cu
constexpr int kRemRows = 32;
// attention_packed.cu: those remainders, packed across groups into 128-row tiles that walk over all keys with
// per-row route masks.  rem_pos / rem_grp [BH][N], rem_cnt [BH] are built from the query offsets and the routes once per
// plan (groups that route alike are neighbours in the list).
cudaError_t init_attention_packed();
void launch_remainder_rows(const int* q_off, const int* route_ptr, const int* route_idx, int BH, int Cq, int Ck, int N, int* rem_pos,
                           int* rem_grp, int* rem_cnt, cudaStream_t st);
bool launch_attention_packed(const AttnArgs& a, const int* rem_pos, const int* rem_grp, const int* rem_cnt, cudaStream_t st);
// one warp runs the bounded mbarrier wait into its limit (2^16 cycles) and records SPARSEPR_ERR_TIMEOUT in *err
void launch_selftest_bounded_wait(int* err, cudaStream_t st);
// correction_tc.cu: O <- X + X A + c in place, X = O + O_lo (two bf16 words, O_lo [BH][N][128] contiguous), d_v = 128;
// At: bf16 scratch [2][BH][128][128] (the map as two bf16 words)
cudaError_t init_correction_tc();
bool launch_correction_tc(const float* A, const float* c, __nv_bfloat16* At, const void* O_lo, void* O, const i64* os, int BH,
                          int H, int N, int* err, cudaStream_t st);

struct ProbeArgs {
  int dtype, BH, H, N, d, M, Ck, Cq, n_split;
  int kv_div;                          // query heads per K/V head; Kg, Vg, kv_off are indexed by bh / kv_div
  float scale;
  const void *Q; i64 qs[3];            // original layout (probe rows are gathered by index)
  const void *Kg, *Vg;                 // group-major [BH][N][d]
  const int *probe_idx, *q_assign, *kv_off, *route_ptr, *route_idx;
  float* partial;                      // [BH][n_split][M][2][d+2]
  float *X, *Dn;                       // outputs [BH][M][d]: sparse and dense rows
};
size_t probe_partial_floats(int BH, int n_split, int M, int d);
void launch_probe_rows(const ProbeArgs& a, cudaStream_t st);
void launch_probe_merge(const ProbeArgs& a, cudaStream_t st);
// probe_tc.cu: the same partial states from the tensor-core kernel (bf16, d = 128); Qp: scratch [BH][M][128] bf16
cudaError_t init_probe_tc();
bool probe_tc_supported(const ProbeArgs& a);
bool launch_probe_rows_tc(const ProbeArgs& a, __nv_bfloat16* Qp, int* err, cudaStream_t st);
void launch_write_probe_rows(int dtype, const float* Dn, const int* probe_idx, int BH, int H, int M, int d, void* O,
                             const i64* os, cudaStream_t st);

// ---- fit.cu -----------------------------------------------------------------------
struct FitArgs {
  int BH, M, d, r_out;
  bool full_rank;                      // r_out >= min(M, d): Psi Psi^T acts as the identity, no eigenvectors are computed
  float lambda, eps_std;
  bool precise;                        // float64 eigen-solver for the subspace
  const float *X, *Dn, *w;             // [BH][M][d], [BH][M][d], [BH][M]
  double* scratch;                     // see fit_scratch_doubles
  double* eig_ws;                      // eig_scratch_doubles(BH, d) doubles
  float *A, *c;                        // outputs [BH][d][d], [BH][d]
  float* Psi;                          // [BH][d][r] scratch
  int* err;
};
size_t fit_scratch_doubles(int BH, int M, int d);
cudaError_t init_fit();
void launch_fit(const FitArgs& a, cudaStream_t st);

}  // namespace spr
