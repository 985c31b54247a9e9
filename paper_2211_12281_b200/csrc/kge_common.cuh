// Shared declarations of the sm_100a KGE library: host handle, workspace layout, small
// device helpers.  Internal to the library (the public surface is include/kge.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>

#include "../../include/kge.h"
#include "kge_device_once.h"

namespace kge {

constexpr int kMaxDim = 512;     // floats per entity row
constexpr int kCandCap = 1024;   // top-k candidate slots per query between two selections

// Arithmetic shape of a pair (query b, tail n) once the per-query vector q_b is built.
enum Kind : int {
    KIND_L1 = 0,     // TransE p=1:            -sum_k |q_k - t_k|
    KIND_L2 = 1,     // TransE / RotatE p=2:   -sqrt(sum_k (q_k - t_k)^2)
    KIND_CL1 = 2,    // RotatE p=1:            -sum_k |q_k - t_k| over complex moduli
    KIND_DOT = 3,    // DistMult / ComplEx:    sum_k q_k t_k
    KIND_TH_L1 = 4,  // TransH p=1:            x = (q - t) + (w.t) w per pair
    KIND_TH_L2 = 5   // TransH p=2
};

inline Kind kind_of(const kge_config& c) {
    switch (c.score) {
        case KGE_TRANSE: return c.p_norm == 1 ? KIND_L1 : KIND_L2;
        case KGE_ROTATE: return c.p_norm == 1 ? KIND_CL1 : KIND_L2;
        case KGE_ROTATE_REAL_L1: return c.p_norm == 1 ? KIND_L1 : KIND_L2;   // the same query vector and chain rule, the real norm
        case KGE_TRANSH: return c.p_norm == 1 ? KIND_TH_L1 : KIND_TH_L2;
        default: return KIND_DOT;
    }
}

// Device workspace, carved out of the caller's buffer by kge_bind.
struct Workspace {
    int32_t* status;       // [4] sticky status word + scratch flags
    float* loss;           // [1]
    int32_t* counts;       // [8]  U_ent, U_rel, ...
    // graph (canonical order)
    int32_t *gh, *gr, *gt; // [T]
    int64_t* off;          // [P*P*(R+1)]
    uint64_t* wcum;        // [P*P*(R+1)]
    uint64_t* gstart;      // [P*P*R + 1] on-device preprocessing: triples per key, then first sorted index per key
    uint32_t* ghist;       // [256 * tiles + 1] on-device preprocessing: digit-major tile histograms of a radix pass
    // batch
    int32_t *heads, *rels, *tails, *negs;  // contiguous [3B+N]
    float *Q, *What, *Tneg;                // [B,d], [B,d] (TransH), [N,d]
    float *fpos, *gpos, *Lrow;             // [B]
    // feature-projection encoder (Eq. 1)
    uint16_t *Fb;                          // [2B+N, F] bf16 features of the batch's slots [heads | tails | negs]
    uint16_t *Mb;                          // [2][d, F] bf16 copies of M_H, M_T
    float *proj;                           // [2B+N, d] M e_F of every slot (added to the gathered rows)
    uint16_t *Gslot;                       // [2B+N, d] bf16 copy of the slots' gradient rows
    float *dMpart;                         // [2][splits][d, F] partial gradients of M_H, M_T
    float *reg_s3;                         // [2B+N] sum of |e_k|^3 of the gathered rows [heads | tails | negs] (L3 regulariser), or NULL
    uint16_t *Qb, *Tb;                     // [B,d], [N,d] bf16 copies of Q and Tneg (tensor-core scoring)
    uint16_t *Gb;                          // bf16 [B,ldN] dL/dF (ldN = N rounded up to 8)
    float *Gcol;                           // [N] column sums of dL/dF (TransE p=2 on tensor cores)
    float *stat_part, *row_stat;           // [B, pieces, 4], [B, 2] loss statistics of the fused tensor-core forward
    float *grow_part, *gcol_part;          // [B, pieces], [4*tiles_m, N] partial sums of dL/dF
    float *qn2, *tn2;                      // [B], [N] squared norms of the fp32 rows (TransE p=2 by norm expansion)
    float *Grow;                           // [B] row sums of dL/dF (TransE p=1 backward)
    float *Cpart;                          // [St, N] column sums of dL/dF per row split (TransE p=1 backward)
    float *F;                              // [B,N] scores, overwritten by dL/dF
    float *U, *Cc;                         // [B,N] TransH: w.t and the contraction c' = sum_k s_k w_k of every pair
    float *wsum;                           // [B] TransH: sum of the unit normal's coordinates
    // TransH with the backward's two per-pair-coefficient contractions on tensor cores: bf16 two-term splits
    // (x = x1 + x2 up to 2^-17 relative) of c = -dL/dF c' as [B, 2 Np] = [c1 | c2] (Np = N rounded up to 64,
    // padding kept zero), of the negatives as [N, 2d] = [t1 | t2] and of the unit normals as [B, 2d]
    uint16_t *Csb, *Tsb, *Wsb;
    uint16_t *W3b, *T3b;                   // [B, 3 dp], [N, 3 dp] bf16 three-term splits [x1 | x2 | x3] of normals and negatives (dp = d rounded up to 64, padding zero): operands of u = w.t
    float *dQpart, *dWpart, *dTpart;       // [Sq,B,d], [Sq,B,d] (TransH), [St,N,d]
    float *grad_ent, *grad_rel, *grad_relw;  // [2B+N,d], [B,kw], [B,d]
    // dedup
    int32_t *ent_perm, *ent_sorted, *ent_uniq, *ent_seg;  // [2B+N], [2B+N], [2B+N], [2B+N+1]
    int32_t *rel_perm, *rel_sorted, *rel_uniq, *rel_seg;  // [B] ...
    int32_t *ent_segof, *rel_segof;        // [2B+N], [B] segment index of every sorted position
    int32_t *ent_done, *rel_done, *relw_done;   // [2B+N], [B], [B] finished pieces per long segment
    uint64_t *ent_tkeys, *rel_tkeys;       // tile-sorted (id, position) keys, padded to whole tiles
    float *part_ent, *part_rel, *part_relw;  // [list length, width] partial sums of long segments
    // inference
    double* mrr;                           // [1] mean reciprocal rank of the last kge_eval_mrr (in the header block)
    float *iq, *iwhat, *iftrue;            // [maxq,d], [maxq,d], [maxq]
    uint16_t *iqb, *Eb;                    // [maxq,d], [E,d] bf16 query vectors and entity table (tensor-core inference)
    float *thr;                            // [maxq] current k-th best score (-inf until the list is full)
    int32_t *thr_id;                       // [maxq] its id
    int32_t *cand_cnt, *beat_tmp, *beat;   // [maxq]
    float *cand_score; int32_t *cand_id;   // [maxq, kCandCap]
    float *top_score; int32_t *top_id;     // [maxq, topk] running lists
    int32_t *hq_heads, *hq_rels, *hq_tails, *hq_ranks;   // [maxq] staging of kge_score_all_topk_host
    int32_t *hq_ids; float *hq_scores;                   // [maxq, topk]
};

}  // namespace kge

namespace kge {
// Optional per-stage device timing (kge_profile): CUDA events around each launch.
enum Stage : int {
    ST_SAMPLE = 0, ST_BUILD, ST_BLOCK, ST_LOSS, ST_TH_U, ST_ACCUM_Q, ST_ACCUM_T, ST_CHAIN,
    ST_RANK, ST_SEGMENT, ST_UPDATE, ST_TH_CONTRACT, ST_COUNT
};
struct StageTimer {
    bool on = false, created = false;
    cudaEvent_t a[ST_COUNT], b[ST_COUNT];
    bool used[ST_COUNT] = {};
    double ms[ST_COUNT] = {};
    int64_t n[ST_COUNT] = {};
};
}  // namespace kge

struct kge_handle {
    kge_config cfg;
    kge::StageTimer prof;
    int kw;                 // floats per relation row
    kge::Kind kind;
    float *ent, *rel, *relw, *ent_state, *rel_state, *relw_state;
    char* ws_base;
    size_t ws_bytes;
    kge::Workspace ws;
    int64_t num_triples;
    int32_t max_queries, topk;
    int split_q, split_t;   // column splits of the two backward accumulations
    bool th_tc;             // TransH: sum_n c_bn t_n and sum_b c_bn w_b as tensor-core contractions of bf16 splits
    int th_gsplit;          // K splits of each of those contractions (each leaves two partial slabs)
    bool bound, graph_loaded;
    int64_t launches;
    int num_sms;
    // Side streams and events of the training step: the sort of the touched ids and one of the
    // two backward accumulations run beside the main stream's kernels (created by kge_bind).
    // TMA tensor maps (tensor-core path): Qb, Tb (128-row boxes) for the scores; Gb (128-row boxes) and Tb (64-row boxes,
    // read MN-major) for dQ; Gb and Qb (64-row boxes, read MN-major) for dT
    alignas(64) unsigned char tm_q[128], tm_t[128], tm_g[128], tm_g64[128], tm_t64[128], tm_q64[128];
    alignas(64) unsigned char tm_cs[128], tm_cs64[128], tm_ts64[128], tm_ws64[128], tm_w3[128], tm_t3[128];   // TransH splits: Csb K-major / MN-major, Tsb, Wsb
    alignas(64) unsigned char tm_iq[128], tm_eb[128];   // inference: bf16 query vectors and bf16 entity table
    alignas(64) unsigned char tm_iq32[128], tm_ent32[128];   // inference on CUDA cores: fp32 query vectors and entity table in 64-row x 32-float boxes
    bool tiles32_ready;
    // encoder: features of the head / tail+negative slots and M_H / M_T (K-major, 128-row boxes) for the projection; the
    // slots' gradient rows and features again (MN-major, 64-row boxes) for dM = dE^T . F
    alignas(64) unsigned char tm_fh[128], tm_ft[128], tm_mh[128], tm_mt[128], tm_gh64[128], tm_gt64[128], tm_fh64[128], tm_ft64[128];
    const uint16_t* feat;   // [E, F] bf16 text features (fixed)
    float *MH, *MT, *MH_state, *MT_state;   // [d, F] projection matrices and their optimiser state
    int split_m;            // K splits of the two dM contractions
    bool features_bound;
    bool streams_ready;
    cudaStream_t side[2];
    cudaEvent_t ev_ids, ev_loss, ev_seg, ev_t;
    bool eb_valid;          // the bf16 copy of the entity table (tensor-core inference) matches the table
    int wait_limit;         // tries of every bounded barrier wait in this handle's kernels (kDefaultWaitLimit unless a test shortens it)
    float* capture_scores;  // debug: the training step also writes the B x N score block here (caller's device array), or NULL
    char cuda_err[256];     // text of the last failed CUDA call (a fixed buffer: reporting an error allocates nothing)
};

namespace kge {

constexpr int kDefaultWaitLimit = 1 << 20;   // tries of a bounded barrier wait: seconds in all

#define KGE_CUDA_CHECK(h, expr)                                   \
    do {                                                          \
        cudaError_t e_ = (expr);                                  \
        if (e_ != cudaSuccess) {                                  \
            std::snprintf((h)->cuda_err, sizeof((h)->cuda_err), "%.160s: %s", #expr, cudaGetErrorString(e_)); \
            return KGE_ERR_CUDA;                                  \
        }                                                         \
    } while (0)

#define KGE_LAUNCH_CHECK(h)                                       \
    do {                                                          \
        (h)->launches += 1;                                       \
        cudaError_t e_ = cudaGetLastError();                      \
        if (e_ != cudaSuccess) {                                  \
            std::snprintf((h)->cuda_err, sizeof((h)->cuda_err), "kernel launch: %s", cudaGetErrorString(e_)); \
            return KGE_ERR_CUDA;                                  \
        }                                                         \
    } while (0)

// Runs `set` (a cudaFuncSetAttribute call) once per device: the attribute belongs to the device
// that is current when it is set, so a process that uses several GPUs must set it on each.
template <class F>
inline cudaError_t once_per_device(DeviceOnce& flags, F&& set) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    return static_cast<cudaError_t>(flags.run(dev, set));
}

inline void stage_begin(kge_handle* h, int id, cudaStream_t s) {
    if (h->prof.on) { cudaEventRecord(h->prof.a[id], s); }
}
inline void stage_end(kge_handle* h, int id, cudaStream_t s) {
    if (h->prof.on) { cudaEventRecord(h->prof.b[id], s); h->prof.used[id] = true; }
}
// Synchronises the stream and folds the recorded stage times into the running totals.
int stage_collect(kge_handle* h, cudaStream_t s);

// ---- launch wrappers implemented in the other translation units ----
int launch_sample(kge_handle* h, uint64_t step, int32_t* heads, int32_t* rels, int32_t* tails, int32_t* negs,
                  cudaStream_t s);
// Forward and backward; `side` (or NULL) runs the accumulation over the queries concurrently;
// `dedup_side` (or NULL) gets the sort of the touched ids as soon as the ids are final (the
// caller waits for ev_seg before the update); with `fused_sample` the gather kernel draws the
// batch of `step` itself and leaves the ids in the workspace (heads ... negs must point there).
int launch_forward_backward(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                            const int32_t* negs, float* loss_out, cudaStream_t s, cudaStream_t side, cudaStream_t dedup_side,
                            bool fused_sample, uint64_t step);
// Stable sort of the touched ids, distinct ids and segments (needs only the batch ids).
int launch_dedup(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                 const int32_t* negs, cudaStream_t s);
// Segment sums of the gradient rows and the optimiser step (needs both of the above).
int launch_update(kge_handle* h, uint64_t step, float lr, cudaStream_t s);
// Pieces of the multi-device training step: rows of this shard for a list of ids; one list of (id, gradient row) pairs applied to a table.
int launch_gather_rows(kge_handle* h, const int32_t* ids, int n, int64_t base, float* out, cudaStream_t s);
size_t apply_scratch_bytes(int n, int width);
int launch_apply_gradients(kge_handle* h, float* table, float* state, int64_t rows, int width, const int32_t* ids, const float* grads,
                           int n, uint64_t step, float lr, void* scratch, cudaStream_t s);
// Tensor-core score block: F from the bf16 operand copies; tensor maps are made at bind time.
int tc_make_operand_map(kge_handle* h, void* map_out, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows);
// Tensor map of a row-major fp32 matrix [rows, cols] read in boxes of 64 rows x 32 floats with the 128-byte swizzle.
int tc_make_f32_tile_map(kge_handle* h, void* map_out, const void* base, int64_t rows, int64_t cols);
int tc_backward_tile_cols(int cols);
int tc_pieces_per_tile();
// The dT contraction of the dot-product kinds with a single K split is the negatives' gradient rows: it writes them in place.
bool tc_negatives_direct(const kge_handle* h);
int launch_tc_backward(kge_handle* h, cudaStream_t s, cudaStream_t side);
// TransH score block (scores, w.t, c') and its two backward accumulations (kge_transh.cu).
int launch_th_forward(kge_handle* h, cudaStream_t s);
int launch_th_backward(kge_handle* h, cudaStream_t sq, cudaStream_t st);
int th_contract_slabs(const kge_handle* h);          // partial slabs the tensor-core contractions add per side (0 when off)
int launch_th_contract_gemm(kge_handle* h, cudaStream_t s);
int launch_tc_forward(kge_handle* h, cudaStream_t s);
int launch_tc_gemm_terms(kge_handle* h, const unsigned char* tmA, const unsigned char* tmB, int M, int N, int tstride, float* C,
                         int64_t ldc, cudaStream_t s);
int launch_tc_gemm_nt(kge_handle* h, const unsigned char* tmA, const unsigned char* tmB, int M, int N, int K, float* C, int64_t ldc,
                      cudaStream_t s);
int launch_tc_gemm_tn(kge_handle* h, const unsigned char* tmA64, const unsigned char* tmB64, int M, int N, int K, int split, float* C,
                      int64_t ldc, cudaStream_t s);
// Feature-projection encoder (kge_encoder.cu): M e_F of the batch's slots before the gather; dM and the dense step after the backward.
int encoder_make_maps(kge_handle* h);
int launch_encoder_forward(kge_handle* h, const int32_t* heads, const int32_t* tails, const int32_t* negs, cudaStream_t s);
int launch_encoder_backward(kge_handle* h, uint64_t step, float lr, cudaStream_t s);
int launch_cast_bf16(kge_handle* h, const float* src, uint16_t* dst, int64_t count, cudaStream_t s);
int launch_tc_infer_chunk(kge_handle* h, int nq, int64_t e_lo, int64_t e_hi, const int32_t* true_tails, int64_t id_base, cudaStream_t s);
int dedup_tiles(int n);     // sort tiles of a list of n ids
// On-device graph preprocessing and table initialisation (kge_graph.cu).
size_t graph_hist_words(int64_t num_triples);
int launch_graph_build_device(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails, int64_t n,
                              cudaStream_t s);
int launch_init_table(kge_handle* h, float* out, int64_t rows, int width, float std, int kind, uint32_t stream_id, cudaStream_t s);
// Sharded inference: the bound table holds the entities [ent_base, ent_base + E) of a larger table; query vectors
// (and true-tail scores) were assembled from all shards, ids are global, out_ranks receives the shard's beat counts.
struct ShardScoring { int64_t ent_base; const float* qvec; const float* ftrue; };
int run_score_all_topk(kge_handle* h, const int32_t* qh, const int32_t* qr, int32_t nq, int32_t k,
                       const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                       cudaStream_t s, const ShardScoring* shard = nullptr);
int run_shard_query_vectors(kge_handle* h, const int32_t* qh, const int32_t* qr, int32_t nq, int64_t ent_base, float* qvec_out, cudaStream_t s);
int run_shard_true_scores(kge_handle* h, const float* qvec, const int32_t* qr, const int32_t* true_tails, int32_t nq, int64_t ent_base,
                          float* ftrue_out, cudaStream_t s);
int run_merge_topk(const int32_t* cand_ids, const float* cand_scores, int32_t nq, int32_t per_query, int32_t k, int32_t* out_ids,
                   float* out_scores, cudaStream_t s);

#ifdef __CUDACC__
// ---- device helpers ----
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Records `code` in the sticky status word unless one is already there.
__device__ __forceinline__ void set_status(int32_t* status, int code) { atomicCAS(status, 0, code); }

// Bounds-checked id: an id outside [0, rows) is reported and replaced by row 0.
__device__ __forceinline__ int64_t checked_id(int32_t id, int64_t rows, int32_t* status) {
    if (id < 0 || (int64_t)id >= rows) {
        set_status(status, KGE_ERR_ID_RANGE);
        return 0;
    }
    return id;
}

// ---- asynchronous bulk copies (TMA engine, untiled form) completing on a shared-memory barrier ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(arrivals) : "memory");
}
// Makes freshly initialised barriers visible to the asynchronous proxy; follow with __syncthreads().
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One test of the barrier phase `parity`.  The hardware may park the thread for up to about
// `hint_ns` while the phase is incomplete (it wakes as soon as the phase completes), so a waiting
// thread does not fill its scheduler's issue slots with polls.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t hint_ns = 2000u) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
// Waits for the barrier phase `parity` at most `limit` times (each up to the hint above, then a
// short sleep: seconds in all at the default limit); false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int limit, int spin = 16, unsigned sleep_ns = 256) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > spin) __nanosleep(sleep_ns);
    }
    return false;
}
// The same for a single thread that shares its scheduler with working warps (the copy-issuing and
// MMA-issuing threads of the tensor-core kernel): it sleeps between tests from the first miss on,
// so its polls do not take issue slots from the warps that do the arithmetic.
__device__ __forceinline__ bool mbar_wait_idle(uint64_t* bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(96);
    }
    return false;
}
// dst (shared) and src (global) 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Programmatic dependent launch.  A kernel started with launch_dependent() may become resident
// while the kernel before it in the stream still runs; it must call grid_dependency_wait()
// before it touches anything that kernel (or an earlier one) writes or reads, and everything
// before that call may only set up its own shared memory.  The wait returns once the preceding
// kernels have finished and their writes are visible; with no programmatic edge it returns at
// once.  allow_dependents() lets the next kernel become resident from now on.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float softplusf(float z) { return fmaxf(z, 0.f) + log1pf(expf(-fabsf(z))); }
__device__ __forceinline__ float sigmoidf(float z) {
    if (z >= 0.f) return 1.f / (1.f + expf(-z));
    float e = expf(z);
    return e / (1.f + e);
}
#endif

// Launch with a programmatic edge to the kernel before it in the stream (see grid_dependency_wait).
template <class... P, class... A>
inline cudaError_t launch_dependent(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

}  // namespace kge
