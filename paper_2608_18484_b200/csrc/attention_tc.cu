// Block-sparse / dense attention on the sm_100a tensor cores (bf16, d = d_v = 128).
//
// One CTA processes one 128-row query tile (of one query group, Eq. 3; or of the whole
// head for dense attention, Eq. 1).  Roles:
//   warps 0-7  softmax: warps w and w+4 share the 32 rows of TMEM quadrant w and split the
//              128 scores of a row in two halves (keys 0-63 / 64-127 of the tile)
//   warp  8    TMA producer of Q and the key tiles (+ tile meta ring)
//   warp  9    issues Q K^T (one thread); owns the TMEM allocation
//   warp  10   TMA producer of the value tiles
//   warp  11   issues P V (one thread)
// The routed keys/values arrive as one concatenated sequence of 16-row boxes (tiles of 128 keys, only
// range ends are ragged); consecutive boxes of one key range are fetched by one copy per set bit of their
// number (tensor maps with 16-, 32-, 64- and 128-row boxes).  Data path per key tile i:
//   S_b = Q K_i^T        tcgen05.mma, smem x smem -> TMEM (fp32), two score buffers b = i mod 2; a buffer is
//                        released as soon as the softmax threads hold its scores in registers, so the product
//                        runs two tiles ahead of the softmax
//   P_b = exp2(.)        softmax threads: tcgen05.ld their half row of S_b, row maximum (the two halves meet
//                        through shared memory), bf16 P to TMEM columns of its own (two buffers as well);
//                        3 of every 8 exponentials are a cubic on the FMA pipe, the others use ex2.approx
//   O  += P V_i          tcgen05.mma with the A operand read from TMEM; O stays in TMEM
// A single issuing thread shares its warp scheduler with two softmax warps that rarely leave it an issue slot:
// this is why the two products have a thread each on different schedulers, why the producers issue few, large
// copies, and why the barrier polls of a tile are grouped.
// The reference maximum of a row moves only when it grows by more than 2^8 (then O is rescaled).
// Epilogue: O / l, stored as bf16 at the original token index (inverse permutation).  The residual correction of
// Eq. 9 is a pass of its own (correction_tc.cu) so that the fit can overlap this kernel; for that pass the part of
// every element that the bf16 rounding dropped is stored as a second bf16 word (O_lo), so that the corrected output
// is, in effect, rounded to bf16 only once.
// A tile with at most 64 valid rows (the remainder of a query group) holds every row TWICE, at lanes r and r + 64:
// the softmax threads of lanes 64-127 would otherwise spend a full tile's worth of exponentials on rows that do not
// exist (the loop is bound by the throughput of those instructions).  The four threads that then sit on a row (two
// lanes x two halves) take 32 of its 128 scores each; the copy at lane r accumulates the keys [0,32) and [64,96) of
// every tile, the copy at lane r + 64 the others, and the epilogue adds the two accumulators.  The products
// themselves are unchanged (the tile was padded to 128 rows anyway).
// Every mbarrier wait is bounded; on expiry the CTA records SPARSEPR_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <mutex>
#include "kernels.cuh"
#include "tc_common.cuh"

namespace spr {

namespace tc {

constexpr int kThreads = 384;
constexpr int kTile = 128;            // query rows per CTA, keys per tile
constexpr int kD = 128;
constexpr int kSub = 16;              // rows per TMA box of the K/V stream
constexpr int kSubPerTile = kTile / kSub;
constexpr uint32_t kHalfBytes = kTile * 128;          // one [128 rows x 64 bf16] swizzled block
constexpr uint32_t kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr uint32_t kSubBytes = kSub * 128;            // 2 KB per box
constexpr int kPolyOf8 = 3;            // pairs of every 8 whose exponential is a polynomial on the FMA pipe
constexpr int kKStages = 2;            // K tiles in flight (consumed by Q K^T)
constexpr int kVStages = 2;            // V tiles in flight (consumed by P V)

struct Smem {                          // offsets from a 1024-byte aligned base
  static constexpr uint32_t q = 0;
  static constexpr uint32_t k = q + kTileBytes;
  static constexpr uint32_t v = k + kKStages * kTileBytes;
  static constexpr uint32_t ranges = v + kVStages * kTileBytes;
  static constexpr uint32_t xchg = ranges + kMaxGroups * 8;     // float [2 tile parities][2 halves][128] row maxima; float [2][128] row sums
  static constexpr uint32_t meta = xchg + 6 * 128 * 4;            // uint2[8]: ring of per-tile box counts
  static constexpr uint32_t bars = meta + 8 * 8;                  // kNumBars mbarriers
  static constexpr uint32_t misc = bars + 32 * 8;                 // tmem base, abort flag, counters
  static constexpr uint32_t dst = misc + 64;                      // int [128]: where the rows of this tile go (original token index)
  static constexpr uint32_t total = dst + kTile * 4;
};
constexpr size_t kSmemBytes = Smem::total;                        // the dynamic segment is 1024-byte aligned and the only shared memory

enum Bar { Q_FULL = 0, K_FULL = 1, K_EMPTY = K_FULL + kKStages, V_FULL = K_EMPTY + kKStages, V_EMPTY = V_FULL + kVStages,
           S_FULL = V_EMPTY + kVStages, S_FREE = S_FULL + 2, P_FULL = S_FREE + 2, P_EMPTY = P_FULL + 2, O_DONE = P_EMPTY + 2, META_FULL,
           kNumBars = META_FULL + 8 };
static_assert(kNumBars <= 32, "barrier area");

struct Params {
  int BH, H, N, Cq, Ck, sparse;
  int kv_div;                      // query heads per K/V head: K/V tensors, their maps and kv_off are indexed by head / kv_div
  float scale_log2;
  const int *q_off, *kv_off, *route_ptr, *route_idx, *q_perm, *tile_off;
  __nv_bfloat16* O; i64 os[3];
  float* O_sparse;
  __nv_bfloat16* O_lo;             // optional [BH][N][128]: o - bf16(o), original order (second word for the correction pass)
  int* err;
};

struct Maps { CUtensorMap m[4]; };      // the same tensor with boxes of 16, 32, 64 and 128 rows

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) { return pack_bf16x2(a, b); }

__global__ void __launch_bounds__(kThreads, 1)
k_attention_tc(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapQ64,
               const __grid_constant__ Maps mapsK, const __grid_constant__ Maps mapsV, Params prm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* sm = smem_raw;
  int2* ranges = reinterpret_cast<int2*>(sm + Smem::ranges);
  float* xmax = reinterpret_cast<float*>(sm + Smem::xchg);                 // [2][2][128] half-row maxima of the current / next tile
  float* xsum = xmax + 4 * 128;                                            // [2][128] half-row sums (end)
  uint2* meta = reinterpret_cast<uint2*>(sm + Smem::meta);
  volatile int* misc = reinterpret_cast<volatile int*>(sm + Smem::misc);   // [0] tmem base, [1] abort, [2] total boxes, [3] leave, [4] query group, [5] its first tile
  const uint32_t bars = base + Smem::bars;
  auto bar = [&](int i) { return bars + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, b = bh / prm.H, h = bh % prm.H;
  // ---- which query tile ---------------------------------------------------------------
  // Few dependent global reads: one round finds the query group of this tile (every thread tests one group),
  // reads the error word and stages the key-group offsets in shared memory (the K ring is still idle); the
  // second round reads the group's rows and routes.
  // Once any CTA has recorded a timeout the remaining CTAs of the launch leave at once (also if the
  // shared-memory base is not aligned as the swizzled tiles require).
  int* kv_stage = reinterpret_cast<int*>(sm + Smem::k);
  if (tid == 0) {
    misc[3] = (prm.err != nullptr && *reinterpret_cast<volatile int*>(prm.err) == SPARSEPR_ERR_TIMEOUT) || (base & 1023u) != 0;
    if ((base & 1023u) != 0) set_error(prm.err, SPARSEPR_ERR_CUDA);
    misc[4] = -1;
  }
  __syncthreads();
  if (prm.sparse) {
    const int* toff = prm.tile_off + (i64)bh * (prm.Cq + 1);
    const int* kvo = prm.kv_off + (i64)(bh / prm.kv_div) * (prm.Ck + 1);
    for (int g = tid; g < prm.Cq; g += kThreads)
      if (toff[g] <= (int)blockIdx.x && (int)blockIdx.x < toff[g + 1]) { misc[4] = g; misc[5] = toff[g]; }
    for (int g = tid; g <= prm.Ck; g += kThreads) kv_stage[g] = kvo[g];
    __syncthreads();
  }
  if (misc[3] || (prm.sparse && misc[4] < 0)) return;        // error, or a tile index beyond this head's tiles
  int row0, nrows, nroute;
  const int* ridx = nullptr;
  if (prm.sparse) {
    const int g = misc[4];
    const int* qoff = prm.q_off + (i64)bh * (prm.Cq + 1);
    const int* rp = prm.route_ptr + (i64)bh * (prm.Cq + 1);
    const int q0 = qoff[g], q1 = qoff[g + 1], r0 = rp[g], r1 = rp[g + 1];
    row0 = q0 + ((int)blockIdx.x - misc[5]) * kTile;
    nrows = min(kTile, q1 - row0);
    ridx = prm.route_idx + (i64)bh * prm.Cq * prm.Ck + r0;
    nroute = r1 - r0;
  } else {
    row0 = blockIdx.x * kTile;
    nrows = min(kTile, prm.N - row0);
    nroute = 1;
  }
  const bool dup = prm.sparse && nrows <= kTile / 2;           // every row twice: lanes r and r + 64 (see the header)
  // destination rows of the tile, fetched now so that the epilogue does not wait for them
  int* dsts = reinterpret_cast<int*>(sm + Smem::dst);
  if (tid < kTile) dsts[tid] = tid < nrows ? (prm.sparse ? prm.q_perm[(i64)bh * prm.N + row0 + tid] : row0 + tid) : -1;

  // ---- set-up: barriers, TMEM, key ranges ---------------------------------------------------
  if (tid == 0) {
    for (int i = 0; i < kNumBars; ++i)
      mbar_init(bar(i), (i == P_FULL || i == P_FULL + 1 || i == S_FREE || i == S_FREE + 1) ? 256 : 1);
    misc[1] = 0; misc[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(base + Smem::misc, 512);
  __syncthreads();
  {
    int boxes = 0;
    for (int t = tid; t < nroute; t += kThreads) {
      int start = 0, len = prm.N;
      if (prm.sparse) { const int g = ridx[t]; start = kv_stage[g]; len = kv_stage[g + 1] - start; }
      ranges[t] = make_int2(start, len);
      boxes += (len + kSub - 1) / kSub;
    }
    boxes = warp_sum(boxes);
    if (lane == 0 && boxes) atomicAdd((int*)&misc[2], boxes);
  }
  fence_async_smem();                        // the staged offsets were read from memory that the copies will overwrite
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = (uint32_t)misc[0];
  const int total_boxes = misc[2];
  const int n_tiles = (total_boxes + kSubPerTile - 1) / kSubPerTile;
  volatile int* abort_flag = &misc[1];

  if (warp == 8 || warp == 10) {
    // =========================== TMA producers ==========================================
    // warp 8 streams Q and the key tiles, warp 10 the value tiles.  All lanes of a producer walk
    // the concatenated key ranges together (uniform); lane j issues the copies of box j.
    if (n_tiles > 0) {
      const bool is_k = warp == 8;
      const int c3 = prm.sparse ? 0 : b;
      const int c2 = (prm.sparse ? bh : h) / prm.kv_div;       // K/V head (group-major copies: [BH / kv_div]; originals: [B][H / kv_div])
      if (is_k && lane == 0) {
        const int q2 = prm.sparse ? bh : h;
        mbar_expect_tx(bar(Q_FULL), kTileBytes);
        if (dup) {
          // the same 64 rows into both halves of the tile (rows 64-127 of a [128 x 64] block start 8 KB in)
          for (int part = 0; part < 2; ++part) {
            tma_load_4d(base + Smem::q + part * (kHalfBytes / 2), &mapQ64, bar(Q_FULL), 0, row0, q2, c3);
            tma_load_4d(base + Smem::q + kHalfBytes + part * (kHalfBytes / 2), &mapQ64, bar(Q_FULL), 64, row0, q2, c3);
          }
        } else {
          tma_load_4d(base + Smem::q, &mapQ, bar(Q_FULL), 0, row0, q2, c3);
          tma_load_4d(base + Smem::q + kHalfBytes, &mapQ, bar(Q_FULL), 64, row0, q2, c3);
        }
      }
      const int nst = is_k ? kKStages : kVStages;
      const int full0 = is_k ? K_FULL : V_FULL, empty0 = is_k ? K_EMPTY : V_EMPTY;
      const uint32_t buf0 = base + (is_k ? Smem::k : Smem::v);
      const Maps* maps = is_k ? &mapsK : &mapsV;
      int ri = 0, off = 0;
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % nst;
        const uint32_t ph = ((i / nst) & 1) ^ 1;             // empty barriers: the first pass completes immediately
        // the tile takes up to 8 boxes of 16 rows; consecutive boxes of one key range form a segment, and a segment
        // of n boxes is fetched by one copy per set bit of n (128, 64, 32 or 16 rows), largest first
        int my_start = 0, my_t = 0, my_n = 0, nsub = 0;
        uint32_t cnt_bits = 0;
        while (nsub < kSubPerTile && ri < nroute) {
          const int2 rg = ranges[ri];
          const int left = rg.y - off, nb = (left + kSub - 1) / kSub;
          const int n = min(kSubPerTile - nsub, nb);
          if (lane >= nsub && lane < nsub + n) { my_t = lane - nsub; my_n = n; my_start = rg.x + off + my_t * kSub; }
          uint32_t bits = n == 8 ? 0xFFFFFFFFu : ((1u << (4 * n)) - 1u);      // valid rows of every box, minus one
          if (n == nb) {                                                       // the range ends here: its last box may be short
            const int sh = 4 * (n - 1);
            bits = (bits & ~(0xFu << sh)) | ((uint32_t)(left - (n - 1) * kSub - 1) << sh);
            ++ri; off = 0;
          } else {
            off += n * kSub;
          }
          cnt_bits |= bits << (4 * nsub);
          nsub += n;
        }
        int my_k = -1;                                                         // log2 of the boxes this lane's copy spans
#pragma unroll
        for (int kb = 0; kb < 4; ++kb)
          if (lane < nsub && ((my_n >> kb) & 1) && my_t == ((my_n >> (kb + 1)) << (kb + 1))) my_k = kb;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(empty0 + s), ph, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          if (is_k) {
            // the key producer runs at most four tiles ahead of the last reader of meta[i]: ring of 8
            meta[i & 7] = make_uint2(cnt_bits, (uint32_t)nsub);
            mbar_arrive(bar(META_FULL + (i & 7)));
          }
          mbar_expect_tx(bar(full0 + s), nsub * 2 * kSubBytes);
        }
        __syncwarp();
        if (my_k >= 0) {
          const uint32_t dst = buf0 + s * kTileBytes + lane * kSubBytes;
          tma_load_4d(dst, &maps->m[my_k], bar(full0 + s), 0, my_start, c2, c3);
          tma_load_4d(dst + kHalfBytes, &maps->m[my_k], bar(full0 + s), 64, my_start, c2, c3);
        }
      }
    }
  } else if (warp == 9) {
    // =========================== Q K^T issuer ============================================
    // TMEM columns: S_0 [0,128), S_1 [128,256), P_0 [256,320) and P_1 [448,512) (two bf16 per column), O [320,448).
    // The two products are issued by two threads on different warp schedulers: an issuing thread shares its
    // scheduler with two softmax warps that rarely leave it a slot, and the score tile two steps ahead must not
    // queue behind the P V of the current one.
    if (lane == 0 && n_tiles > 0) {
      const uint32_t idesc_qk = idesc_bf16(0, 128);
      // descriptors are built once; inside the loops only their address field moves (in 16-byte units)
      const uint64_t q_desc = smem_desc(base + Smem::q, 16);
      const uint64_t k_desc0 = smem_desc(base + Smem::k, 16);
      bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kKStages;
        // score buffer i mod 2 is free once every softmax thread holds tile i - 2 in registers
        if (i >= 2 && !mbar_wait(bar(S_FREE + (i & 1)), ((i - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(K_FULL + s), (i / kKStages) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem + (uint32_t)(i & 1) * 128u;
        const uint64_t kd = k_desc0 + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint64_t koff = (uint64_t)((kk >> 2) * (kHalfBytes >> 4) + (kk & 3) * 2);     // compile-time constant
          umma_bf16(d, q_desc + koff, kd + koff, idesc_qk, kk > 0);
        }
        umma_commit(bar(K_EMPTY + s));
        umma_commit(bar(S_FULL + (i & 1)));
      }
    }
  } else if (warp == 11) {
    // =========================== P V issuer ==============================================
    if (lane == 0 && n_tiles > 0) {
      const uint32_t idesc_pv = idesc_bf16(1, 128);
      const uint64_t v_desc0 = smem_desc(base + Smem::v, kHalfBytes);
      bool ok = true;
      for (int i = 0; i < n_tiles && ok; ++i) {
        const int s = i % kVStages;
        if (!mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag)) { ok = false; break; }
        const int nsub = (int)meta[i & 7].y;
        if (!mbar_wait(bar(V_FULL + s), (i / kVStages) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar(P_FULL + (i & 1)), (i >> 1) & 1, abort_flag)) { ok = false; break; }   // P(i) in TMEM, O rescaled if needed
        tc_fence_after();
        const uint32_t d = tmem + 320u;
        const uint32_t pa = tmem + ((i & 1) ? 448u : 256u);
        const uint64_t vd = v_desc0 + (uint64_t)(s * (kTileBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < kSubPerTile; ++kk)
          if (kk < nsub)
            umma_bf16_ts(d, pa + kk * 8, vd + (uint64_t)(kk * (kSubBytes >> 4)), idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bar(V_EMPTY + s));
        umma_commit(bar(P_EMPTY + (i & 1)));
      }
      if (ok) umma_commit(bar(O_DONE));
    }
  } else if (warp < 8) {
    // =========================== softmax (warps 0-7) =======================================
    // Thread (half hh, quadrant wq, lane) owns the 64 scores of keys [64 hh, 64 hh + 64) of query row
    // 32 wq + lane; warps wq and wq + 4 meet at the named barrier 1 + wq to agree on the row maximum.
    const int hh = warp >> 2, wq = warp & 3;
    const int row = wq * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t FULL = 0xffffffffu;
    const uint32_t p_addr0 = tmem + lane_addr + 256u + (uint32_t)hh * 32u;      // P of even tiles; odd tiles 192 columns on
    const uint32_t o_addr = tmem + lane_addr + 320u + (uint32_t)hh * 64u;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    const float sc = prm.scale_log2;
    // the 64 finished output columns [64 hh, 64 hh + 64) of tile row r: bf16 at the original token index, the part that
    // the rounding dropped as a second word, float32 on request
    auto store_row = [&](int r, const float (&o)[64]) {
      const int dst = prm.sparse ? prm.q_perm[(i64)bh * prm.N + row0 + r] : row0 + r;
      __nv_bfloat16* op = prm.O + b * prm.os[0] + h * prm.os[1] + (i64)dst * prm.os[2] + hh * 64;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        float v8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k];
        store8(op + ch * 8, v8);
      }
      if (prm.O_lo) {                                          // what the bf16 rounding above dropped
        __nv_bfloat16* lp = prm.O_lo + ((i64)bh * prm.N + dst) * kD + hh * 64;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          float v8[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k] - __bfloat162float(__float2bfloat16_rn(o[ch * 8 + k]));
          store8(lp + ch * 8, v8);
        }
      }
      if (prm.O_sparse) {
        float* sp = prm.O_sparse + ((i64)bh * prm.N + dst) * kD + hh * 64;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          float v8[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) v8[k] = o[ch * 8 + k];
          store8(sp + ch * 8, v8);
        }
      }
    };
    if (dup) {
      // ================= at most 64 valid rows: four threads per row, 32 scores each ==================
      const int u = wq >> 1, q0 = wq & 1;                        // copy of the row (lane r or r + 64); pair of quadrants
      const int vr = q0 * 32 + lane;                             // the row, 0..63
      const int cb = 64 * hh + 32 * u;                           // this thread's keys of a tile: [cb, cb + 32)
      const int slot = 2 * hh + u;
      for (int i = 0; i < n_tiles; ++i) {
        const bool t_meta = mbar_try(bar(META_FULL + (i & 7)), (i >> 3) & 1);
        const bool t_s = mbar_try(bar(S_FULL + (i & 1)), (i >> 1) & 1);
        const bool t_pe = i > 1 ? mbar_try(bar(P_EMPTY + (i & 1)), ((i - 2) >> 1) & 1) : true;
        {
          bool w = ok;
          if (!t_meta) w = w && mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag);
          if (!t_s) w = w && mbar_wait(bar(S_FULL + (i & 1)), (i >> 1) & 1, abort_flag);
          ok = __all_sync(FULL, w);
        }
        float s[32];
        float mx = -INFINITY;
        if (ok) {
          tc_fence_after();
          const uint2 mt = meta[i & 7];
          tmem_ld32_nowait(tmem + lane_addr + (uint32_t)(i & 1) * 128u + (uint32_t)cb, s);
          tmem_ld_wait();
          tc_fence_before();
          mbar_arrive(bar(S_FREE + (i & 1)));                       // the scores are in registers
          if (!(mt.x == 0xFFFFFFFFu && mt.y == 8u)) {
#pragma unroll
            for (int bx = 0; bx < 2; ++bx) {
              const int box = (cb >> 4) + bx;
              const int lim = box < (int)mt.y ? (int)((mt.x >> (4 * box)) & 15u) : -1;    // last valid column of the box
              if (lim != 15) {
#pragma unroll
                for (int c = 0; c < 16; ++c) s[bx * 16 + c] = (c <= lim) ? s[bx * 16 + c] : -INFINITY;
              }
            }
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            mx4[0] = max3(mx4[0], s[c], s[c + 1]); mx4[1] = max3(mx4[1], s[c + 2], s[c + 3]);
            mx4[2] = max3(mx4[2], s[c + 4], s[c + 5]); mx4[3] = max3(mx4[3], s[c + 6], s[c + 7]);
          }
          mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        }
        // the four threads of a row exchange their maxima (four warps meet: both halves of quadrants q0 and q0 + 2)
        float* xm = xmax + (i & 1) * 256;
        xm[slot * 64 + vr] = mx;
        asm volatile("bar.sync %0, 128;" ::"r"(1 + q0) : "memory");
        mx = fmaxf(fmaxf(xm[vr], xm[64 + vr]), fmaxf(xm[128 + vr], xm[192 + vr]));
        const bool move = (mx - m_ref) * sc > 8.f;
        const float m_new = move ? mx : m_ref;
        const float corr = move ? ex2((m_ref - m_new) * sc) : 1.f;
        const float mneg = -m_new * sc;
        m_ref = m_new;
        if (!__all_sync(FULL, t_pe)) {
          ok = __all_sync(FULL, ok && (t_pe || mbar_wait(bar(P_EMPTY + (i & 1)), ((i - 2) >> 1) & 1, abort_flag)));
          tc_fence_after();
        }
        if (!ok) continue;
        if (i > 0 && __any_sync(FULL, move)) {                   // rescale this half of the lane's accumulator (rare)
          ok = __all_sync(FULL, mbar_wait(bar(P_EMPTY + ((i - 1) & 1)), ((i - 1) >> 1) & 1, abort_flag));
          if (!ok) continue;
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            float t[32];
            tmem_ld32(o_addr + q * 32, t);
#pragma unroll
            for (int c = 0; c < 32; ++c) t[c] *= corr;
            tmem_st32(o_addr + q * 32, t);
          }
        }
        float2 ps2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        const float2 sc2 = make_float2(sc, sc), mneg2 = make_float2(mneg, mneg);
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          float2 x = __ffma2_rn(make_float2(s[2 * q], s[2 * q + 1]), sc2, mneg2);
          if ((q & 7) < kPolyOf8) x = ex2_poly2(x);
          else { x.x = ex2(x.x); x.y = ex2(x.y); }
          s[2 * q] = x.x; s[2 * q + 1] = x.y;
          ps2[q & 1] = __fadd2_rn(ps2[q & 1], x);
        }
        l = l * corr + ((ps2[0].x + ps2[0].y) + (ps2[1].x + ps2[1].y));
        // P of this lane and half: this thread's 32 probabilities -> 16 columns, zeros in the 16 columns of the keys
        // that the other copy of the row takes
        {
          uint32_t w[16], z[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) { w[c] = pack_bf16(s[2 * c], s[2 * c + 1]); z[c] = 0u; }
          const uint32_t pa = p_addr0 + (uint32_t)(i & 1) * 192u;
          tmem_st16u_nowait(pa + 16u * (uint32_t)u, w);
          tmem_st16u_nowait(pa + 16u * (uint32_t)(1 - u), z);
          tmem_st_wait();
        }
        tc_fence_before();
        mbar_arrive(bar(P_FULL + (i & 1)));
      }
      // ---- row sums of the four threads, sum of the two accumulators, normalise, store -----------------
      if (n_tiles > 0) ok = __all_sync(FULL, ok && mbar_wait(bar(O_DONE), 0, abort_flag));
      xsum[slot * 64 + vr] = l;
      float o[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) o[c] = 0.f;
      if (ok && n_tiles > 0) {
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float t[32];
          tmem_ld32(o_addr + q * 32, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) o[q * 32 + c] = t[c];
        }
      }
      // the copy at lane r + 64 hands its accumulator over through the Q tile's shared memory (every product that
      // reads it has completed): [half][column][row], conflict-free for consecutive rows
      float* ex = reinterpret_cast<float*>(sm + Smem::q);
      if (u == 1) {
#pragma unroll
        for (int c = 0; c < 64; ++c) ex[(hh * 64 + c) * 64 + vr] = o[c];
      }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + q0) : "memory");
      if (u == 0) {
        const float ltot = (xsum[vr] + xsum[64 + vr]) + (xsum[128 + vr] + xsum[192 + vr]);
        const float inv = ltot > 0.f ? 1.f / ltot : 0.f;
#pragma unroll
        for (int c = 0; c < 64; ++c) o[c] = inv != 0.f ? (o[c] + ex[(hh * 64 + c) * 64 + vr]) * inv : 0.f;
        if (ok && vr < nrows) store_row(vr, o);
      }
    } else {
    for (int i = 0; i < n_tiles; ++i) {
      // the three barriers of this tile are polled back to back (their shared-memory round trips overlap); the P
      // buffer of this parity was consumed by the product two tiles back and is normally free long before
      const bool t_meta = mbar_try(bar(META_FULL + (i & 7)), (i >> 3) & 1);
      const bool t_s = mbar_try(bar(S_FULL + (i & 1)), (i >> 1) & 1);
      const bool t_pe = i > 1 ? mbar_try(bar(P_EMPTY + (i & 1)), ((i - 2) >> 1) & 1) : true;
      {
        bool w = ok;
        if (!t_meta) w = w && mbar_wait(bar(META_FULL + (i & 7)), (i >> 3) & 1, abort_flag);
        if (!t_s) w = w && mbar_wait(bar(S_FULL + (i & 1)), (i >> 1) & 1, abort_flag);
        ok = __all_sync(FULL, w);
      }
      float s[64];
      float mx = -INFINITY;
      if (ok) {
        tc_fence_after();
        const uint2 mt = meta[i & 7];
        const uint32_t s_addr = tmem + lane_addr + (uint32_t)(i & 1) * 128u + (uint32_t)hh * 64u;
        tmem_ld32_nowait(s_addr, *reinterpret_cast<float(*)[32]>(&s[0]));
        tmem_ld32_nowait(s_addr + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(bar(S_FREE + (i & 1)));                         // the scores are in registers
        if (!(mt.x == 0xFFFFFFFFu && mt.y == 8u)) {
          // only the boxes that end a key range (or lie beyond the stream) have columns to mask; the test is uniform
#pragma unroll
          for (int bx = 0; bx < 4; ++bx) {
            const int box = hh * 4 + bx;
            const int lim = box < (int)mt.y ? (int)((mt.x >> (4 * box)) & 15u) : -1;      // last valid column of the box
            if (lim != 15) {
#pragma unroll
              for (int c = 0; c < 16; ++c) s[bx * 16 + c] = (c <= lim) ? s[bx * 16 + c] : -INFINITY;
            }
          }
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 64; c += 8) {
          mx4[0] = max3(mx4[0], s[c], s[c + 1]); mx4[1] = max3(mx4[1], s[c + 2], s[c + 3]);
          mx4[2] = max3(mx4[2], s[c + 4], s[c + 5]); mx4[3] = max3(mx4[3], s[c + 6], s[c + 7]);
        }
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      }
      // the two halves of the row exchange their maxima (buffer of this tile's parity; executed whatever happened)
      float* xm = xmax + (i & 1) * 256;
      xm[hh * 128 + row] = mx;
      asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
      mx = fmaxf(mx, xm[(hh ^ 1) * 128 + row]);
      const bool move = (mx - m_ref) * sc > 8.f;                 // true on the first tile (m_ref = -inf); same in both halves
      const float m_new = move ? mx : m_ref;
      const float corr = move ? ex2((m_ref - m_new) * sc) : 1.f; // 0 on the first tile
      const float mneg = -m_new * sc;
      m_ref = m_new;
      // the P buffer of this parity must have been consumed by the product two tiles back
      if (!__all_sync(FULL, t_pe)) {
        ok = __all_sync(FULL, ok && (t_pe || mbar_wait(bar(P_EMPTY + (i & 1)), ((i - 2) >> 1) & 1, abort_flag)));
        tc_fence_after();
      }
      if (!ok) continue;                                         // warp-uniform; the pair barrier above has been passed
      if (i > 0 && __any_sync(FULL, move)) {                     // rescale this half of the warp's O rows (rare)
        // O must be at rest: the product of the previous tile has to be complete as well
        ok = __all_sync(FULL, mbar_wait(bar(P_EMPTY + ((i - 1) & 1)), ((i - 1) >> 1) & 1, abort_flag));
        if (!ok) continue;
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float t[32];
          tmem_ld32(o_addr + q * 32, t);
#pragma unroll
          for (int c = 0; c < 32; ++c) t[c] *= corr;
          tmem_st32(o_addr + q * 32, t);
        }
      }
      // exponentials: kPolyOf8 of every 8 pairs on the FMA pipe, the others on the special-function unit
      float2 ps2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 sc2 = make_float2(sc, sc), mneg2 = make_float2(mneg, mneg);
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        float2 x = __ffma2_rn(make_float2(s[2 * q], s[2 * q + 1]), sc2, mneg2);
        if ((q & 7) < kPolyOf8) x = ex2_poly2(x);
        else { x.x = ex2(x.x); x.y = ex2(x.y); }
        s[2 * q] = x.x; s[2 * q + 1] = x.y;
        ps2[q & 1] = __fadd2_rn(ps2[q & 1], x);
      }
      l = l * corr + ((ps2[0].x + ps2[0].y) + (ps2[1].x + ps2[1].y));
      // P (bf16, two per 32-bit column): this half's 64 probabilities -> 32 columns
      {
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) w[c] = pack_bf16(s[2 * c], s[2 * c + 1]);
        tmem_st32u(p_addr0 + (uint32_t)(i & 1) * 192u, w);
      }
      tc_fence_before();
      mbar_arrive(bar(P_FULL + (i & 1)));
    }
    // ---- row sums of the two halves, normalise, store ------------------------------------------
    if (n_tiles > 0) ok = __all_sync(FULL, ok && mbar_wait(bar(O_DONE), 0, abort_flag));
    xsum[hh * 128 + row] = l;
    asm volatile("bar.sync %0, 64;" ::"r"(1 + wq) : "memory");
    const float ltot = l + xsum[(hh ^ 1) * 128 + row];
    const float inv = ltot > 0.f ? 1.f / ltot : 0.f;
    // this thread finishes output columns [64 hh, 64 hh + 64) of its row
    float o[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) o[c] = 0.f;
    if (ok && n_tiles > 0) {
      tc_fence_after();
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        float t[32];
        tmem_ld32(o_addr + q * 32, t);
#pragma unroll
        for (int c = 0; c < 32; ++c) o[q * 32 + c] = inv != 0.f ? t[c] * inv : 0.f;
      }
    }
    if (prm.O_sparse) {
      if (ok && row < nrows) store_row(row, o);
    } else {
      // Coalesced stores: a thread holds 64 columns of one row, and storing them directly makes every 16-byte store
      // of a warp touch 32 different lines.  The tile is staged in shared memory instead (the K and V rings are idle:
      // every product has completed), rows 272 bytes apart so that the 16-byte accesses of a quarter warp fall into
      // different banks, and written out with 16 lanes per row.
      constexpr uint32_t kPitch = 2 * kD + 16;
      unsigned char* st_hi = sm + Smem::k;
      unsigned char* st_lo = sm + Smem::v;
      {
        uint4* ph = reinterpret_cast<uint4*>(st_hi + row * kPitch + hh * 128);
        uint4* pl = reinterpret_cast<uint4*>(st_lo + row * kPitch + hh * 128);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          uint32_t wh[4], wl[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float a0 = o[ch * 8 + 2 * k], a1 = o[ch * 8 + 2 * k + 1];
            wh[k] = pack_bf16(a0, a1);
            wl[k] = pack_bf16(a0 - __bfloat162float(__float2bfloat16_rn(a0)), a1 - __bfloat162float(__float2bfloat16_rn(a1)));
          }
          ph[ch] = make_uint4(wh[0], wh[1], wh[2], wh[3]);
          if (prm.O_lo) pl[ch] = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        }
      }
      asm volatile("bar.sync 6, 256;" ::: "memory");
      const int c16 = lane & 15;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int r = warp * 16 + 2 * it + (lane >> 4);
        const int dst = dsts[r];
        if (ok && r < nrows) {
          const uint4 vh = *reinterpret_cast<const uint4*>(st_hi + r * kPitch + c16 * 16);
          *reinterpret_cast<uint4*>(prm.O + b * prm.os[0] + h * prm.os[1] + (i64)dst * prm.os[2] + c16 * 8) = vh;
          if (prm.O_lo) {
            const uint4 vl = *reinterpret_cast<const uint4*>(st_lo + r * kPitch + c16 * 16);
            *reinterpret_cast<uint4*>(prm.O_lo + ((i64)bh * prm.N + dst) * kD + c16 * 8) = vl;
          }
        }
      }
    }
    }
  }
  // ---- teardown ----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
    if (tid == 0) set_error(prm.err, SPARSEPR_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---- tensor maps (driver entry point fetched through the runtime; libcuda is not linked) -------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_encode_once;

EncodeTiledFn encode_fn() {
  std::call_once(g_encode_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  });
  return g_encode;
}

bool tma_available() { return encode_fn() != nullptr; }

bool make_map(CUtensorMap* m, const void* ptr, int cols, int rows, int H, int B, i64 sb, i64 sh, i64 sn, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const i64 hstride = H > 1 ? sh : (i64)rows * sn;
  const i64 bstride = B > 1 ? sb : (i64)H * hstride;
  const cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)H, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)hstride * 2, (cuuint64_t)bstride * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

cudaError_t init_attention_tc() {
  return cudaFuncSetAttribute(tc::k_attention_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes);
}

bool attention_tc_supported(const AttnArgs& a) {
  return a.dtype == SPARSEPR_BF16 && a.d == 128 && tc::tma_available();
}

bool launch_attention_tc(const AttnArgs& a, cudaStream_t st) {
  using namespace tc;
  CUtensorMap mq, mq64;
  Maps mk, mv;
  const bool sparse = a.route_ptr != nullptr;
  const int B = a.BH / a.H;
  const int kvd = a.kv_div < 1 ? 1 : a.kv_div;
  bool ok;
  if (sparse) {
    ok = make_map(&mq, a.Q, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kTile) &&
         make_map(&mq64, a.Q, kD, a.N, a.BH, 1, 0, (i64)a.N * kD, kD, kTile / 2);
    for (int k = 0; k < 4 && ok; ++k)
      ok = make_map(&mk.m[k], a.K, kD, a.N, a.BH / kvd, 1, 0, (i64)a.N * kD, kD, kSub << k) &&
           make_map(&mv.m[k], a.V, kD, a.N, a.BH / kvd, 1, 0, (i64)a.N * kD, kD, kSub << k);
  } else {
    ok = make_map(&mq, a.Q, kD, a.N, a.H, B, a.qs[0], a.qs[1], a.qs[2], kTile) &&
         make_map(&mq64, a.Q, kD, a.N, a.H, B, a.qs[0], a.qs[1], a.qs[2], kTile / 2);
    for (int k = 0; k < 4 && ok; ++k)
      ok = make_map(&mk.m[k], a.K, kD, a.N, a.H / kvd, B, a.ks[0], a.ks[1], a.ks[2], kSub << k) &&
           make_map(&mv.m[k], a.V, kD, a.N, a.H / kvd, B, a.vs[0], a.vs[1], a.vs[2], kSub << k);
  }
  if (!ok) return false;
  Params p{};
  p.BH = a.BH; p.H = a.H; p.N = a.N; p.Cq = a.Cq; p.Ck = a.Ck; p.sparse = sparse; p.kv_div = kvd;
  p.scale_log2 = a.scale * 1.4426950408889634f;
  p.q_off = a.q_off; p.kv_off = a.kv_off; p.route_ptr = a.route_ptr; p.route_idx = a.route_idx; p.q_perm = a.q_perm;
  p.tile_off = a.tile_off;
  p.O = (__nv_bfloat16*)a.O; for (int i = 0; i < 3; ++i) p.os[i] = a.os[i];
  p.O_sparse = a.O_sparse; p.O_lo = (__nv_bfloat16*)a.O_lo; p.err = a.err;
  const int tiles = (a.N + kTile - 1) / kTile + (sparse ? a.Cq : 0);
  k_attention_tc<<<dim3(tiles, a.BH), kThreads, kSmemBytes, st>>>(mq, mq64, mk, mv, p);
  return true;
}

}  // namespace spr
