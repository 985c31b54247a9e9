// Tensor-core score block (5th-generation tensor cores: tcgen05.mma with the accumulator in
// tensor memory, operands staged in shared memory by TMA tensor copies).
//
//   C[M, N] = A[M, K] . B[N, K]^T      A, B bf16, K contiguous; fp32 accumulation
//
// Persistent CTAs (one per SM) each walk a run of 128 x 128 output tiles.  Warp 0 feeds a ring of
// shared-memory stages with TMA (one elected lane), warp 1 issues the MMAs (one elected lane)
// into one of two accumulators in tensor memory and owns the allocation, warps 2-17 drain the
// other accumulator meanwhile (a warp may only touch the 32 lanes of its own quarter; four warps
// share a quarter, a quarter of the columns each) and apply the epilogue:
//   EPI_STORE   C = acc (the backward contractions)
//   EPI_STATS   no score leaves the chip: per row and 64-column piece the running maximum, the sum
//               of exponentials and the weighted loss sum of Section 3.1 "Loss Functions"; the
//               score is the contraction (DistMult, ComplEx) or, for TransE with p = 2, the
//               norm expansion -sqrt(max(|q|^2 + |t|^2 - 2 acc, 0))
//   EPI_GRAD    scores recomputed, dL/dF formed from the finished row statistics and written as
//               bf16 in both orientations for the two backward contractions
// Every wait on a barrier is bounded; a wait that runs out records KGE_ERR_TIMEOUT, tells the
// other warps to stop, and the CTA still releases its tensor memory before it returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "kge_common.cuh"

namespace kge {

namespace {

constexpr int TC_BM = 128, TC_BN = 128, TC_BK = 64;      // BK bf16 = one 128-byte swizzle row
constexpr int TC_STAGES = 4;
constexpr int TC_RING_MAX = 8;                            // barriers are laid out for the deepest ring (resident column tile, below)
constexpr int TC_EPI_WARPS = 8;                           // epilogue warps of the training kernels: TC_EPI_GROUPS per tensor-memory lane quarter
constexpr int TC_EPI_WARPS_TOPK = 16;                     // the filter epilogue of full-entity scoring profits from more
constexpr int TC_EPI_GROUPS = TC_EPI_WARPS / 4;
constexpr int TC_GRAD_STAGE_BYTES = 2048;                 // per epilogue warp: 32 rows x 32 bf16 columns on their way to memory
constexpr int TC_STORE_STAGE_BYTES = 4096;                // the same for EPI_STORE's 32 rows x 32 fp32 columns
constexpr int TC_PIECE = TC_BN / TC_EPI_GROUPS;           // columns of a 128-wide tile per piece of loss statistics
// The fused loss epilogues on 256-column tiles run on sixteen warps as well (64 columns = one piece of statistics per warp):
// measured against eight, C3 passes 41.5 / 58.0 -> 39.4 / 53.8 us, the special-function-bound C4 passes 98.7 / 154.7 -> 98.9 / 135.8 us,
// although sixteen warps leave 96 registers per thread and the norm-expansion variants spill a little.
constexpr int TC_FUSED_WARPS_256 = 16;
__host__ __device__ constexpr int tc_epi_warps(int epi, int bn = 128) {   // 3 = EPI_TOPK, 1 / 2 = the fused loss epilogues
    return (epi & 3) == 3 ? TC_EPI_WARPS_TOPK : ((((epi & 3) == 1 || (epi & 3) == 2) && bn == 256) ? TC_FUSED_WARPS_256 : TC_EPI_WARPS);
}
__host__ __device__ constexpr int tc_threads(int epi, int bn = 128) { return 32 * (2 + tc_epi_warps(epi, bn)); }
constexpr uint32_t TC_A_BYTES = TC_BM * TC_BK * 2;
constexpr uint32_t TC_MN_GROUP_BYTES = 64 * TC_BK * 2;    // MN-major operand: 64 contiguous elements x 64 K rows per TMA box
__host__ __device__ constexpr uint32_t tc_stage_bytes(int bn) { return TC_A_BYTES + (uint32_t)bn * TC_BK * 2; }
__host__ __device__ constexpr size_t tc_smem_bytes(int bn) { return 1024 + (size_t)TC_STAGES * tc_stage_bytes(bn) + 256; }
constexpr int TC_BEAT_ROWS_MAX = 8 * 1024;                 // queries whose rank counts fit in shared memory beside the 256-column stages

enum { EPI_STORE = 0, EPI_STATS = 1, EPI_GRAD = 2, EPI_TOPK = 3, EPI_L2 = 4, EPI_CE = 8,    // L2 / CE: flags of the fused loss epilogues
       EPI_A1 = 16 };   // log-sigmoid loss of a distance score with self-adversarial temperature exactly 1 (see tc_stats_chunk)

struct TcGemmParams {
    int M, N, K;
    int kb_per_split;                     // 64-wide slices of K per split
    int tiles_m, tiles_n, items;          // items = splits * tiles_m * tiles_n
    int bn;                               // columns per tile (128 or 256)
    float* C; int64_t ldc;
    int64_t split_stride;                 // floats between the output slabs of consecutive K splits
    const float *row_norm2, *col_norm2;   // norm expansion: |q_b|^2 [M], |t_n|^2 [N]
    int32_t* status;
    int wait_limit;                       // tries of a bounded barrier wait
    // fused loss epilogues (EPI_STATS, EPI_GRAD): the score is acc, or for l2 != 0 the distance score above
    int l2, loss;
    float gamma, adv_temp, ce_c, loss_scale;
    int row_pieces;                       // pieces of TC_PIECE columns per row of stat_part / grow_part
    float4* stat_part;                    // [M, row_pieces] per column piece: (max, sum exp, weighted loss sum, -)
    const float2* row_stat;               // [M] (max, 1 / normaliser) of the whole row
    uint16_t* Gb; int64_t ldg;            // [M, ldg] bf16 dL/dF (divided by the distance for l2)
    float* grow_part;                     // [M, row_pieces] sums of the written values per column piece
    float* gcol_part;                     // [4 * tiles_m, N] sums per 32-row piece (l2 only)
    // full-entity scoring (EPI_TOPK): rows are queries, columns the entities [n_base, n_base + N)
    int m_fastest;                        // walk the row tiles of one column tile first (the column tile stays in L2)
    int64_t n_base;
    int64_t id_base;                      // the caller's id of table row 0 (sharded inference)
    const float *thr, *ftrue;             // [M] current k-th best score; score of the true tail
    const int32_t *thr_id, *tt;           // [M] its id; true tail ids (or NULL)
    int32_t *cand_cnt, *beat_tmp;         // [M] candidates appended in this chunk; entities ordered before the true tail
    float* cand_score; int32_t* cand_id;  // [M, cand_cap]
    int cand_cap;
    int32_t* overflow;                    // set when a candidate list is full
    int beat_rows;                        // rows whose rank counts are gathered in shared memory first (0: global atomics)
    int resident_b;                       // EPI_TOPK: the column tile has a buffer of its own and the ring holds row tiles only
};

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile written by TMA with the 128-byte
// swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart, tile base 1024-byte aligned.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                          // leading byte offset (not used by swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                          // layout type: 128-byte swizzle
    return d;
}

// The same for an operand whose M (or N) index is the contiguous one ("MN-major"), as TMA leaves
// it from boxes of 64 contiguous elements x 64 K rows: inside a box a K row is 128 bytes, groups
// of 8 K rows are 1024 bytes apart (stride offset), the next 64 elements of M / N are one box
// (8192 bytes) further (leading offset).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(TC_MN_GROUP_BYTES >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor: D fp32, A and B bf16, M x N tile; a_mn / b_mn: that operand is MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n, bool a_mn = false, bool b_mn = false) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
// (the registers are valid after tmem_ld_wait)
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) { tmem_ld32_issue(taddr, v); tmem_ld_wait(); }

struct TcItem { int z, m0, n0; };   // K split, first row, first column

constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
__device__ __forceinline__ float fast_exp2(float y) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y)); return r; }
__device__ __forceinline__ float fast_log2(float y) { float r; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y)); return r; }
__device__ __forceinline__ float fast_rcp(float y) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y)); return r; }
__device__ __forceinline__ float fast_rsqrt(float y) { float r; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y)); return r; }

// The fused epilogues evaluate one transcendental per special-function instruction: their
// inputs come from bf16 operands, so the approximate forms (relative error about 2^-22) are
// far inside the error of the scores, and an epilogue of a d = 128 contraction is bound by
// exactly these instructions.
// softplus(z) = max(z, 0) + log(1 + exp(-|z|))
__device__ __forceinline__ float tc_softplus(float z) {
    const float e = fast_exp2(-fabsf(z) * kLog2e);
    return fmaf(fast_log2(1.f + e), kLn2, fmaxf(z, 0.f));
}
// sigmoid(z) from the same exponential
__device__ __forceinline__ float tc_sigmoid(float z) {
    const float e = fast_exp2(-fabsf(z) * kLog2e);
    const float r = fast_rcp(1.f + e);
    return z >= 0.f ? r : e * r;
}

// Score of a pair from the accumulator: the contraction itself, or (L2) the distance score of
// the norm expansion, with the reciprocal distance the gradient needs (0 at distance 0).
template <bool L2>
__device__ __forceinline__ float tc_score_inv(const TcGemmParams& p, float acc, float rn, int col, float& inv) {
    if (!L2) { inv = 0.f; return acc; }
    const float s2 = fmaxf(rn + p.col_norm2[col] - 2.f * acc, 0.f);
    inv = s2 > 0.f ? fast_rsqrt(s2) : 0.f;
    return -s2 * inv;
}
template <bool L2>
__device__ __forceinline__ float tc_score(const TcGemmParams& p, float acc, float rn, int col) {
    float inv;
    return tc_score_inv<L2>(p, acc, rn, col, inv);
}


// Per-row inputs of an epilogue, read before the accumulator is waited for.
struct TcRowState {
    float rn;                 // squared norm of the row (norm expansion)
    float2 st;                // EPI_GRAD: the row's (base-2 maximum, 1 / normaliser)
    float thr, ft;            // EPI_TOPK: current k-th best score, score of the true tail
    int32_t thr_id, tt;       //           its id, the true tail's id
};
template <int EPI>
__device__ __forceinline__ TcRowState tc_row_state(const TcGemmParams& p, int row) {
    TcRowState r{0.f, make_float2(0.f, 0.f), INFINITY, 0.f, 0, -1};
    if (row >= p.M) return r;   // rows outside the problem: no true tail, a threshold nothing exceeds
    if ((EPI & EPI_L2) != 0) r.rn = p.row_norm2[row];
    if ((EPI & 3) == EPI_GRAD) r.st = p.row_stat[row];
    if ((EPI & 3) == EPI_TOPK) {
        r.thr = p.thr[row]; r.thr_id = p.thr_id[row];
        if (p.tt) { r.ft = p.ftrue[row]; r.tt = p.tt[row]; }
    }
    return r;
}

// One chunk of 32 scores of the first pass.  FULL: all 32 columns lie inside the problem (no
// per-element masking); otherwise the first `valid` do.
// A1 (distance scores f <= 0, log-sigmoid loss, temperature a = 1): the weight exponential and the loss term share one
// exponential.  With e = 2^(y - m) the weight term, exp(gamma + f) = K e with K = exp(gamma) 2^m (one special-function
// instruction per chunk and lane; K <= exp(gamma) because f <= 0), and softplus(gamma + f) = log(1 + K e): three
// special-function instructions per score (distance, exponential, logarithm) instead of four.
template <bool L2, bool CE, bool FULL, bool A1 = false>
__device__ __forceinline__ void tc_stats_chunk(const TcGemmParams& p, float (&v)[32], float rn, int ncol, int valid,
                                               float k1, float k0, float& m, float& z, float& l) {
    // four independent chains each for the maximum and the sums: a single chain of 32 dependent
    // operations would leave the few epilogue warps waiting on their own results
    float cmv[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        if (L2) v[i] = (FULL || i < valid) ? tc_score<true>(p, v[i], rn, ncol + i) : 0.f;
        const float y = fmaf(v[i], k1, k0);        // exponent in base 2
        if (CE) v[i] = y;                          // the sampled softmax does not need the score itself again
        cmv[i & 3] = fmaxf(cmv[i & 3], (FULL || i < valid) ? y : -INFINITY);
    }
    const float cm = fmaxf(fmaxf(cmv[0], cmv[1]), fmaxf(cmv[2], cmv[3]));
    if (cm > m) { const float r = fast_exp2(m - cm); z *= r; l *= r; m = cm; }
    float zv[4] = {0.f, 0.f, 0.f, 0.f}, lv[4] = {0.f, 0.f, 0.f, 0.f};
    const float kexp = A1 ? fast_exp2(fmaf(p.gamma, kLog2e, m)) : 0.f;      // exp(gamma) 2^m
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float e = fast_exp2((CE ? v[i] : fmaf(v[i], k1, k0)) - m);
        if (!FULL && i >= valid) e = 0.f;
        zv[i & 3] += e;
        if (A1) lv[i & 3] = fmaf(e, kLn2 * fast_log2(fmaf(kexp, e, 1.f)), lv[i & 3]);
        else if (!CE) lv[i & 3] = fmaf(e, tc_softplus(p.gamma + v[i]), lv[i & 3]);
    }
    z += (zv[0] + zv[1]) + (zv[2] + zv[3]);
    if (!CE) l += (lv[0] + lv[1]) + (lv[2] + lv[3]);
}

// First pass of the fused loss: running (max, sum of exponentials, exponentially weighted loss
// sum) over this thread's 64 columns of one row, rescaled whenever the maximum moves.  The
// exponent is x = a f for the self-adversarial weights and x = f + c for the sampled softmax;
// it is carried in base 2 (y = x log2 e), so an exponential is one ex2 of a difference.
template <bool L2, bool CE, bool A1>
__device__ __forceinline__ void tc_epilogue_stats(const TcGemmParams& p, const TcItem& it, int row, const TcRowState& rs, int col_off, uint32_t taddr) {
    const float rn = rs.rn;
    const float k1 = CE ? kLog2e : p.adv_temp * kLog2e, k0 = CE ? p.ce_c * kLog2e : 0.f;
    float m = -INFINITY, z = 0.f, l = 0.f;
    static_assert(TC_PIECE == 64, "two chunks of 32 columns per piece");
    float v0[32], v1[32];
    tmem_ld32_issue(taddr, v0);                // both chunks are requested before the first is used
    tmem_ld32_issue(taddr + 32u, v1);
    tmem_ld_wait();
    if (row < p.M) {
        const int ncol = it.n0 + col_off;
        const int valid0 = min(32, p.N - ncol), valid1 = min(32, p.N - ncol - 32);   // columns inside the problem (may be <= 0)
        if (valid0 == 32) tc_stats_chunk<L2, CE, true, A1>(p, v0, rn, ncol, valid0, k1, k0, m, z, l);
        else if (valid0 > 0) tc_stats_chunk<L2, CE, false, A1>(p, v0, rn, ncol, valid0, k1, k0, m, z, l);
        if (valid1 == 32) tc_stats_chunk<L2, CE, true, A1>(p, v1, rn, ncol + 32, valid1, k1, k0, m, z, l);
        else if (valid1 > 0) tc_stats_chunk<L2, CE, false, A1>(p, v1, rn, ncol + 32, valid1, k1, k0, m, z, l);
    }
    const int piece = (it.n0 + col_off) / TC_PIECE;
    if (row < p.M && piece < p.row_pieces) p.stat_part[(int64_t)row * p.row_pieces + piece] = make_float4(m, z, l, 0.f);
}

__device__ __forceinline__ float bf16_value(uint16_t bits) { return __uint_as_float((uint32_t)bits << 16); }

// dL/dF of one pair from its accumulator: scale = loss_scale / normaliser, k0 already holds minus
// the row's base-2 maximum.
// A1: sigmoid(gamma + f) = t / (1 + t) with t = exp(gamma + f) = krow e, e the weight exponential 2^(y - max) and
// krow = exp(gamma) 2^max per row: one reciprocal instead of an exponential and a reciprocal.
template <bool L2, bool CE, bool A1>
__device__ __forceinline__ float tc_grad_one(const TcGemmParams& p, float acc, float rn, int col, float k1, float k0, float scale, float krow) {
    float inv;
    const float f = tc_score_inv<L2>(p, acc, rn, col, inv);
    const float e = fast_exp2(fmaf(f, k1, k0));
    float g = scale * e;
    if (A1) { const float t = krow * e; g *= t * fast_rcp(1.f + t); }
    else if (!CE) g *= tc_sigmoid(p.gamma + f);
    if (L2) g *= inv;
    return g;
}

// Second pass: dL/dF from the recomputed score and the row's final (base-2 max, 1 / normaliser),
// written as bf16 for the two backward contractions (which read it K-major and MN-major).
// A warp's 32 rows x 32 columns of bf16 pass through `stage` (2 KB of shared memory of its own)
// on their way out, so that a store instruction writes whole 32-byte sectors: eight rows x 64
// contiguous bytes instead of 16 bytes in each of 32 rows.  The 16-byte chunk c of row r sits at
// chunk c ^ ((r >> 1) & 3) of the row: both the row-wise writes and the 8-row reads then touch
// every bank once.
template <bool L2, bool CE, bool A1>
__device__ __forceinline__ void tc_epilogue_grad(const TcGemmParams& p, const TcItem& it, int row, const TcRowState& rs, int col_off, uint32_t taddr,
                                                 uint4* stage) {
    const bool rin = row < p.M;
    const float rn = rs.rn;
    const float2 st = rs.st;
    const float k1 = CE ? kLog2e : p.adv_temp * kLog2e, k0 = (CE ? p.ce_c * kLog2e : 0.f) - st.x;
    const float scale = p.loss_scale * st.y;
    const float krow = A1 ? fast_exp2(fmaf(p.gamma, kLog2e, st.x)) : 0.f;     // exp(gamma) 2^(row maximum)
    const int lane = threadIdx.x & 31;
    float rsum = 0.f;
#pragma unroll 1
    for (int c0 = col_off; c0 < col_off + TC_PIECE; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + (uint32_t)(c0 - col_off), v);
        const int ncol = it.n0 + c0;
        const int valid = rin ? min(32, p.N - ncol) : 0;
        uint32_t g2[16];     // bf16 pairs in memory order
        if (valid == 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = tc_grad_one<L2, CE, A1>(p, v[i], rn, ncol + i, k1, k0, scale, krow);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = i < valid ? tc_grad_one<L2, CE, A1>(p, v[i], rn, ncol + i, k1, k0, scale, krow) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 pr = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            g2[i] = *reinterpret_cast<const uint32_t*>(&pr);
        }
        if (ncol + 32 <= p.N) {       // warp-uniform: all 32 columns lie inside the problem
            const int sw = (lane >> 1) & 3;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                stage[lane * 4 + (i ^ sw)] = make_uint4(g2[4 * i], g2[4 * i + 1], g2[4 * i + 2], g2[4 * i + 3]);
            __syncwarp();
            const int row0 = row - lane;             // first of this warp's 32 rows
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = i * 8 + (lane >> 2), c = lane & 3;
                const uint4 val = stage[r * 4 + (c ^ ((r >> 1) & 3))];
                if (row0 + r < p.M) *reinterpret_cast<uint4*>(p.Gb + (int64_t)(row0 + r) * p.ldg + ncol + c * 8) = val;
            }
            __syncwarp();
        } else if (valid > 0) {
            uint16_t* dst = p.Gb + (int64_t)row * p.ldg + ncol;
#pragma unroll
            for (int i = 0; i < 32; ++i) if (i < valid) dst[i] = (uint16_t)(g2[i >> 1] >> ((i & 1) * 16));
        }
        if (L2) {   // the norm expansion also needs the sums of what the contractions will see
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                v[i] = bf16_value((uint16_t)(g2[i >> 1] >> ((i & 1) * 16)));
                rsum += v[i];
            }
            // Sums over this warp's 32 rows (rows outside the problem hold zeros) of all 32 columns
            // at once: each exchange halves the columns a lane still carries, so 31 shuffles do
            // what 32 separate warp sums need 160 for; lane c ends with the sum of column c.
#pragma unroll
            for (int half = 16; half >= 1; half >>= 1) {
                const bool upper = (lane & half) != 0;
#pragma unroll
                for (int j = 0; j < half; ++j) {
                    const float send = upper ? v[j] : v[j + half], keep = upper ? v[j + half] : v[j];
                    v[j] = keep + __shfl_xor_sync(0xffffffffu, send, half);
                }
            }
            if (ncol + lane < p.N)
                p.gcol_part[(int64_t)((it.m0 / TC_BM) * 4 + ((row - it.m0) >> 5)) * p.N + ncol + lane] = v[0];
        }
    }
    const int piece = (it.n0 + col_off) / TC_PIECE;
    if (L2 && rin && piece < p.row_pieces) p.grow_part[(int64_t)row * p.row_pieces + piece] = rsum;
}

// 1.0f if a > b, else 0.0f, in one instruction.
__device__ __forceinline__ float one_if_gt(float a, float b) {
    float r;
    asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
// Maximum of three in one instruction.
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Largest float below x (x finite or -inf; -inf maps to itself).
__device__ __forceinline__ float float_below(float x) {
    if (x == 0.f) return __uint_as_float(0x80000001u);
    if (x == -INFINITY) return x;
    const uint32_t b = __float_as_uint(x);
    return __uint_as_float(x > 0.f ? b - 1u : b + 1u);
}

// Full-entity scoring (Section 3.1 "Inference"): a score survives into the query's candidate
// list if it is ordered before the query's current k-th best under (score descending, entity
// id ascending); entities ordered before the true tail are counted for its rank.
// Within a run of 32 consecutive entity ids that does not contain the reference id, "ordered
// before (f0, id0)" is a plain comparison: f >= f0 if the run lies below id0, f > f0 if above;
// f >= f0 is written f > (largest float below f0).  Only the run that contains the reference
// id takes the element-by-element form, so the common case costs a compare-and-count per score
// for the rank and one maximum per score for the candidate test.
template <int WIDTH>
__device__ __forceinline__ void tc_epilogue_topk(const TcGemmParams& p, const TcItem& it, int row, const TcRowState& rs, int col_off, uint32_t taddr, int32_t* beat_sm) {
    const bool rin = row < p.M;
    // rows outside the problem stay in the loop (the warp votes below need every lane): their state
    // holds no true tail and a threshold nothing exceeds
    const float thr = rs.thr, ft = rs.ft; const int32_t thr_id = rs.thr_id, tt = rs.tt;
    const float thr_lo = float_below(thr), ft_lo = float_below(ft);
    const int lane = threadIdx.x & 31;
    int beat = 0;
    auto chunk = [&](float (&v)[32], int c0) {
        const int ncol = it.n0 + c0;
        const int valid = min(32, p.N - ncol);          // the same for every lane
        if (valid <= 0) return;
        const int32_t e0 = (int32_t)(p.n_base + p.id_base + ncol);
        if (valid != 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i) if (i >= valid) v[i] = -INFINITY;   // never counted, never a candidate
        }
        // rank of the true tail.  The branch is taken by the whole warp (a vote), so that the
        // element-by-element form stays out of the instruction stream of the common case.
        if (p.tt) {
            const bool inside = tt >= e0 && tt < e0 + 32;
            if (!__any_sync(0xffffffffu, inside)) {
                // counted in floating point (exact: at most 8 per chain) on four independent chains:
                // the comparison yields 1.0f and the additions go to the FMA pipe
                const float c = tt >= e0 + 32 ? ft_lo : ft;
                float n[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int i = 0; i < 32; ++i) n[i & 3] += one_if_gt(v[i], c);
                if (tt >= 0) beat += (int)((n[0] + n[1]) + (n[2] + n[3]));
            } else if (tt >= 0) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int32_t e = e0 + i;
                    if (e != tt && (v[i] > ft || (v[i] == ft && e < tt))) ++beat;
                }
            }
        }
        // candidates: anything ordered before the current k-th best
        float vm[4];           // a tree of three-input maxima, not a chain of 31
#pragma unroll
        for (int j = 0; j < 4; ++j)
            vm[j] = max3(max3(v[8 * j], v[8 * j + 1], v[8 * j + 2]), max3(v[8 * j + 3], v[8 * j + 4], v[8 * j + 5]), fmaxf(v[8 * j + 6], v[8 * j + 7]));
        const float vmax = fmaxf(max3(vm[0], vm[1], vm[2]), vm[3]);
        // Rare once the threshold has tightened, but one warp of the sixteen that share a tile
        // meets it at most tiles, and the tile waits for its slowest warp.  So the warp takes the
        // flagged lanes one at a time and spreads that lane's 32 scores over its 32 lanes (one
        // shuffle per score): the ordering test and the append then run once per lane, not 32
        // times in a row.
        unsigned pending = __ballot_sync(0xffffffffu, vmax > thr_lo);
        while (pending) {
            const int src = __ffs(pending) - 1;
            pending &= pending - 1;
            float f = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float t = __shfl_sync(0xffffffffu, v[i], src);
                if (lane == i) f = t;
            }
            const float thr_s = __shfl_sync(0xffffffffu, thr, src);
            const int32_t id_s = __shfl_sync(0xffffffffu, thr_id, src);
            const int row_s = __shfl_sync(0xffffffffu, row, src);
            const int32_t e = e0 + lane;
            if (f > thr_s || (f == thr_s && e < id_s && f != -INFINITY)) {     // (padded columns hold -inf and never pass)
                const int slot = atomicAdd(&p.cand_cnt[row_s], 1);
                if (slot < p.cand_cap) {
                    p.cand_score[(int64_t)row_s * p.cand_cap + slot] = f;
                    p.cand_id[(int64_t)row_s * p.cand_cap + slot] = e;
                } else {
                    *p.overflow = 1;   // the host redoes this chunk in pieces that cannot overflow
                }
            }
        }
    };
    static_assert(WIDTH % 64 == 0, "two chunks of 32 columns are requested from tensor memory at a time");
#pragma unroll 1
    for (int c0 = col_off; c0 < col_off + WIDTH; c0 += 64) {
        float v0[32], v1[32];
        tmem_ld32_issue(taddr + (uint32_t)(c0 - col_off), v0);
        tmem_ld32_issue(taddr + (uint32_t)(c0 - col_off) + 32u, v1);
        tmem_ld_wait();
        chunk(v0, c0);
        chunk(v1, c0 + 32);
    }
    if (rin && beat > 0) {
        if (row < p.beat_rows) atomicAdd(&beat_sm[row], beat); else atomicAdd(&p.beat_tmp[row], beat);
    }
}

// Epilogue of one warp on one item: WIDTH columns [col_off, col_off + WIDTH) of the tile row held by
// this thread's tensor-memory lane (taddr points at the first of them).
template <int EPI, int WIDTH>
__device__ __forceinline__ void tc_epilogue(const TcGemmParams& p, const TcItem& it, int row, const TcRowState& rs, int col_off, uint32_t taddr, int32_t* beat_sm) {
    static_assert((EPI & 3) == EPI_STORE || (EPI & 3) == EPI_TOPK || WIDTH % TC_PIECE == 0, "the fused loss epilogues work on pieces of TC_PIECE columns");
    if ((EPI & 3) == EPI_STATS || (EPI & 3) == EPI_GRAD) {
#pragma unroll 1
        for (int c = 0; c < WIDTH; c += TC_PIECE) {
            if ((EPI & 3) == EPI_STATS) tc_epilogue_stats<(EPI & EPI_L2) != 0, (EPI & EPI_CE) != 0, (EPI & EPI_A1) != 0>(p, it, row, rs, col_off + c, taddr + (uint32_t)c);
            else tc_epilogue_grad<(EPI & EPI_L2) != 0, (EPI & EPI_CE) != 0, (EPI & EPI_A1) != 0>(p, it, row, rs, col_off + c, taddr + (uint32_t)c, reinterpret_cast<uint4*>(beat_sm));
        }
        return;
    }
    if ((EPI & 3) == EPI_TOPK) { tc_epilogue_topk<WIDTH>(p, it, row, rs, col_off, taddr, beat_sm); return; }
    float* const Cout = p.C + (int64_t)it.z * p.split_stride;
    const float rn = rs.rn;
#pragma unroll 1
    for (int c0 = col_off; c0 < col_off + WIDTH; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + (uint32_t)(c0 - col_off), v);
        const int ncol = it.n0 + c0;
        if (EPI & EPI_L2) {   // the debug tap of the score block: the distance score of the norm expansion, as the fused epilogues form it
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = ncol + i < p.N ? tc_score<true>(p, v[i], rn, ncol + i) : 0.f;
        }
        if (ncol + 32 <= p.N && (p.ldc & 3) == 0) {
            // (warp-uniform) a lane holds 32 columns of its own row: stored as they are, every instruction would touch
            // 32 rows with 16 bytes each.  Through shared memory (128-byte rows, 16-byte pieces XOR-swizzled by row) an
            // instruction writes four rows' whole 128 bytes.
            float4* st = reinterpret_cast<float4*>(beat_sm);
            const int lane = threadIdx.x & 31, sw = lane & 7, row0 = row - lane;
#pragma unroll
            for (int i = 0; i < 8; ++i) st[lane * 8 + (i ^ sw)] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int r = j * 4 + (lane >> 3), c = lane & 7;
                const float4 val = st[r * 8 + (c ^ (r & 7))];
                if (row0 + r < p.M) *reinterpret_cast<float4*>(Cout + (int64_t)(row0 + r) * p.ldc + ncol + 4 * c) = val;
            }
            __syncwarp();
        } else if (row < p.M) {
            float* dst = Cout + (int64_t)row * p.ldc + ncol;
#pragma unroll
            for (int i = 0; i < 32; ++i) if (ncol + i < p.N) dst[i] = v[i];
        }
    }
}

// Work item = (K split, row tile, column tile), column tile fastest.  A CTA takes a contiguous
// run of items, so consecutive items mostly share their A rows (kept warm in L2).
__device__ __forceinline__ TcItem tc_item(const TcGemmParams& p, int64_t item) {
    if (p.m_fastest) return TcItem{0, (int)(item % p.tiles_m) * TC_BM, (int)(item / p.tiles_m) * p.bn};
    const int tn = (int)(item % p.tiles_n), r = (int)(item / p.tiles_n);
    return TcItem{r / p.tiles_m, (r % p.tiles_m) * TC_BM, tn * p.bn};
}
// The same walk one item at a time: the divisions are paid once per CTA, not once per item and warp.
__device__ __forceinline__ void tc_item_next(const TcGemmParams& p, TcItem& it) {
    if (p.m_fastest) {
        it.m0 += TC_BM;
        if (it.m0 >= p.tiles_m * TC_BM) { it.m0 = 0; it.n0 += p.bn; }
    } else {
        it.n0 += p.bn;
        if (it.n0 >= p.tiles_n * p.bn) {
            it.n0 = 0; it.m0 += TC_BM;
            if (it.m0 >= p.tiles_m * TC_BM) { it.m0 = 0; ++it.z; }
        }
    }
}

// BN: columns per tile (128, or 256 for the backward contractions of wide rows); A_MN / B_MN:
// the operand is read MN-major (its tensor map has the contraction index as rows), which is how
// dL/dF, Q and T serve as transposed operands without a transposed copy.
template <int EPI, int BN = 128, bool A_MN = false, bool B_MN = false>
__global__ void __launch_bounds__(tc_threads(EPI, BN), 1) tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                             const __grid_constant__ CUtensorMap tmB, TcGemmParams p) {
    constexpr uint32_t TC_STAGE_BYTES = tc_stage_bytes(BN);
    constexpr int NACC = 512 / BN;                      // fp32 accumulators in tensor memory, used in turn: all 512 columns
    constexpr uint32_t TC_TMEM_COLS = NACC * BN;
    constexpr int EW = tc_epi_warps(EPI, BN), EG = EW / 4, TC_THREADS = tc_threads(EPI, BN);
    // In the gradient pass of the norm-expansion kinds (bound by special-function instructions, with row- and
    // column-dependent loads) the epilogue warps form two groups that take the CTA's items in turn, so the epilogues
    // of consecutive items overlap: measured faster there (136 against 146 us at B = N = 8192) and slower or equal
    // in every other pass, which stay one group.
    constexpr int EGRP = ((EPI & EPI_L2) != 0 && (EPI & 3) == EPI_GRAD && EG % 2 == 0) ? 2 : 1;
    constexpr int GW = EW / EGRP, GCOLS = BN / (GW / 4);       // warps per group; columns per warp
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* base = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(base + (size_t)TC_STAGES * TC_STAGE_BYTES);
    uint64_t* empty = full + TC_RING_MAX;
    uint64_t* acc_full = empty + TC_RING_MAX;    // [NACC] accumulator buffer written
    uint64_t* acc_empty = acc_full + NACC;       // [NACC] accumulator buffer drained by all epilogue warps
    uint64_t* b_full = acc_empty + NACC;         // resident column tile: loaded / no longer read by any MMA
    uint64_t* b_free = b_full + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_free + 1);
    volatile uint32_t* stop = tmem_slot + 1;     // set by a warp whose wait ran out
    int32_t* beat_sm = reinterpret_cast<int32_t*>(base + (size_t)TC_STAGES * TC_STAGE_BYTES + 256);   // [beat_rows], EPI_TOPK
    if ((EPI & 3) == EPI_TOPK)
        for (int i = threadIdx.x; i < p.beat_rows; i += TC_THREADS) beat_sm[i] = 0;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int per_cta = (p.items + gridDim.x - 1) / gridDim.x;
    const int item_begin = blockIdx.x * per_cta, item_end = min(p.items, item_begin + per_cta);
    const int kb_total = (p.K + TC_BK - 1) / TC_BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_RING_MAX; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(b_full, 1); mbar_init(b_free, 1);
        for (int b = 0; b < NACC; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], GW); }
        *stop = 0;
        mbar_init_fence();
    }
    if (warp == 1) {   // one warp allocates both accumulator buffers and gives up the right to allocate more
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Full-entity scoring with rows of at most 128 coordinates: the column (entity) tile of the
    // current run of items sits in a buffer of its own (2 x 32 KB) and the rest of the stage memory
    // is a ring of eight 16 KB row-tile slices, four items deep.  With the column tile kept inside
    // the ring stages instead, only two items were in flight and the MMAs waited for copies.
    const bool resident = (EPI & 3) == EPI_TOPK && BN == 256 && p.resident_b != 0;
    constexpr uint32_t RES_B_BYTES = 2u * 256u * TC_BK * 2u;          // two slices of the column tile
    constexpr int RES_RING = 8;
    if (warp == 0 && resident) {
        if (lane == 0) {
            int ring = 0, btile = 0, cur_n0 = -1;
            TcItem it = tc_item(p, item_begin);
            for (int item = item_begin; item < item_end && !*stop; ++item, tc_item_next(p, it)) {
                bool ok = true;
                if (it.n0 != cur_n0) {      // a new column tile: every MMA on the previous one must be done
                    cur_n0 = it.n0;
                    ok = mbar_wait_idle(b_free, (btile & 1) ^ 1, p.wait_limit);
                    if (ok) {
                        mbar_arrive_expect_tx(b_full, (uint32_t)kb_total * (256u * TC_BK * 2u));
                        for (int kb = 0; kb < kb_total; ++kb)
#pragma unroll
                            for (int g = 0; g < 2; ++g)
                                tma_load_2d(base + (size_t)kb * (256 * TC_BK * 2) + g * (128 * TC_BK * 2), &tmB, kb * TC_BK,
                                            (int)p.n_base + it.n0 + 128 * g, b_full);
                        ++btile;
                    }
                }
                for (int kb = 0; kb < kb_total && ok; ++kb, ++ring) {
                    const int s = ring % RES_RING;
                    ok = mbar_wait_idle(&empty[s], ((ring / RES_RING) & 1) ^ 1, p.wait_limit);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&full[s], TC_A_BYTES);
                    tma_load_2d(base + RES_B_BYTES + (size_t)s * TC_A_BYTES, &tmA, kb * TC_BK, it.m0, &full[s]);
                }
                if (!ok) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); break; }
            }
        }
    } else if (warp == 1 && resident) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, BN, false, false);
            int ring = 0, btile = 0, cur_n0 = -1;
            bool ok = true;
            TcItem it = tc_item(p, item_begin);
            for (int item = item_begin, local = 0; item < item_end && ok && !*stop; ++item, ++local) {
                const int buf = local % NACC;
                if (it.n0 != cur_n0) {
                    cur_n0 = it.n0;
                    if (!mbar_wait_idle(b_full, btile & 1, p.wait_limit)) { ok = false; break; }
                    ++btile;
                }
                if (!mbar_wait_idle(&acc_empty[buf], ((local / NACC) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)buf * BN;
                for (int kb = 0; kb < kb_total; ++kb, ++ring) {
                    const int s = ring % RES_RING;
                    if (!mbar_wait_idle(&full[s], (ring / RES_RING) & 1, p.wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(base + RES_B_BYTES + (size_t)s * TC_A_BYTES);
                    const uint32_t sb = smem_u32(base + (size_t)kb * (256 * TC_BK * 2));
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        umma_bf16(tmem_acc, umma_desc_k_sw128(sa + k * 32), umma_desc_k_sw128(sb + k * 32), idesc, (kb | k) != 0);
                    umma_commit(&empty[s]);
                }
                umma_commit(&acc_full[buf]);           // also after a failed wait, so the epilogue warps wake up
                tc_item_next(p, it);
                if (item + 1 >= item_end || it.n0 != cur_n0) umma_commit(b_free);   // the last MMAs that read this column tile
            }
            if (!ok) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); }
        }
    } else if (warp == 0) {
        if (lane == 0) {
            int ring = 0;    // slices issued so far: stage = ring % STAGES, phase = ring / STAGES
            // Without K splits and with a slice count that divides the ring, slice kb of every item
            // lands in the same stages, so the operand that consecutive items share (the row tile
            // when column tiles vary fastest, the column tile otherwise) is still there from the item
            // before: it is fetched again only when it changes.  keep[s] = first row (or column) of
            // the shared operand held by stage s.
            const bool reuse = p.kb_per_split == kb_total && TC_STAGES % kb_total == 0;
            int keep[TC_STAGES];
#pragma unroll
            for (int s = 0; s < TC_STAGES; ++s) keep[s] = -1;
            TcItem it = tc_item(p, item_begin);
            for (int item = item_begin; item < item_end && !*stop; ++item, tc_item_next(p, it)) {
                const int kb0 = it.z * p.kb_per_split, nkb = min(p.kb_per_split, kb_total - kb0);
                for (int kb = 0; kb < nkb; ++kb, ++ring) {
                    const int s = ring % TC_STAGES;
                    if (!mbar_wait_idle(&empty[s], ((ring / TC_STAGES) & 1) ^ 1, p.wait_limit)) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); break; }
                    unsigned char* sa = base + (size_t)s * TC_STAGE_BYTES;
                    const int shared_at = p.m_fastest ? it.n0 : it.m0;
                    bool have = false;
#pragma unroll
                    for (int q = 0; q < TC_STAGES; ++q) if (q == s) { have = reuse && keep[q] == shared_at; keep[q] = shared_at; }
                    const bool load_a = !(have && !p.m_fastest), load_b = !(have && p.m_fastest);
                    mbar_arrive_expect_tx(&full[s], (load_a ? TC_A_BYTES : 0u) + (load_b ? TC_STAGE_BYTES - TC_A_BYTES : 0u));
                    const int k0 = (kb0 + kb) * TC_BK;
                    if (!load_a) {
                    } else if (A_MN) {
#pragma unroll
                        for (int g = 0; g < TC_BM / 64; ++g) tma_load_2d(sa + g * TC_MN_GROUP_BYTES, &tmA, it.m0 + 64 * g, k0, &full[s]);
                    } else {
                        tma_load_2d(sa, &tmA, k0, it.m0, &full[s]);
                    }
                    unsigned char* sb = sa + TC_A_BYTES;
                    if (!load_b) {
                    } else if (B_MN) {
#pragma unroll
                        for (int g = 0; g < BN / 64; ++g) tma_load_2d(sb + g * TC_MN_GROUP_BYTES, &tmB, it.n0 + 64 * g, k0, &full[s]);
                    } else {
#pragma unroll
                        for (int g = 0; g < BN / 128; ++g)   // boxes of 128 rows, one after the other
                            tma_load_2d(sb + g * (128 * TC_BK * 2), &tmB, k0, (int)p.n_base + it.n0 + 128 * g, &full[s]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, BN, A_MN, B_MN);
            int ring = 0;
            bool ok = true;
            TcItem it = tc_item(p, item_begin);
            for (int item = item_begin, local = 0; item < item_end && ok && !*stop; ++item, ++local, tc_item_next(p, it)) {
                const int nkb = min(p.kb_per_split, kb_total - it.z * p.kb_per_split);
                const int buf = local % NACC;
                // the epilogue warps must have drained this buffer (two items ago)
                if (!mbar_wait_idle(&acc_empty[buf], ((local / NACC) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)buf * BN;
                for (int kb = 0; kb < nkb; ++kb, ++ring) {
                    const int s = ring % TC_STAGES;
                    if (!mbar_wait_idle(&full[s], (ring / TC_STAGES) & 1, p.wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(base + (size_t)s * TC_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {   // one MMA covers 16 of K: 32 bytes of a K-major row, 16 rows MN-major
                        const uint64_t ad = A_MN ? umma_desc_mn_sw128(sa + k * 2048) : umma_desc_k_sw128(sa + k * 32);
                        const uint64_t bd = B_MN ? umma_desc_mn_sw128(sa + TC_A_BYTES + k * 2048) : umma_desc_k_sw128(sa + TC_A_BYTES + k * 32);
                        umma_bf16(tmem_acc, ad, bd, idesc, (kb | k) != 0);
                    }
                    umma_commit(&empty[s]);            // the stage is free once these MMAs have read it
                }
                umma_commit(&acc_full[buf]);           // also after a failed wait, so the epilogue warps wake up
            }
            if (!ok) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); }
        }
    } else {
        const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
        const int egrp = (warp - 2) / GW;              // which items
        const int cgrp = ((warp - 2) % GW) >> 2;       // which group of the tile's columns
        TcItem it = tc_item(p, min(item_begin + egrp, p.items - 1));
        for (int item = item_begin + egrp, local = egrp; item < item_end; item += EGRP, local += EGRP) {
            if (local != egrp) {
#pragma unroll
                for (int g = 0; g < EGRP; ++g) tc_item_next(p, it);
            }
            // what the epilogue needs of its row does not depend on the accumulator: fetched before the wait
            const TcRowState rs = tc_row_state<EPI>(p, it.m0 + quarter * 32 + lane);
            const int buf = local % NACC;
            const bool ok = mbar_wait_bounded(&acc_full[buf], (local / NACC) & 1, p.wait_limit);
            tc_fence_after();
            if (!ok || *stop) { if (lane == 0) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); } break; }
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cgrp * GCOLS);
            // scratch after the barriers: the rank counts of EPI_TOPK, or 2 / 4 KB per epilogue warp for EPI_GRAD's / EPI_STORE's stores
            int32_t* scratch = (EPI & 3) == EPI_GRAD ? beat_sm + (warp - 2) * (TC_GRAD_STAGE_BYTES / 4)
                             : ((EPI & 3) == EPI_STORE ? beat_sm + (warp - 2) * (TC_STORE_STAGE_BYTES / 4) : beat_sm);
            tc_epilogue<EPI, GCOLS>(p, it, it.m0 + quarter * 32 + lane, rs, cgrp * GCOLS, taddr, scratch);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
    if ((EPI & 3) == EPI_TOPK)     // hand this CTA's rank counts over (integer adds: the result does not depend on the order)
        for (int i = threadIdx.x; i < p.beat_rows; i += TC_THREADS) { const int32_t b = beat_sm[i]; if (b) atomicAdd(&p.beat_tmp[i], b); }
}

// ------------------------------------------------------------------------------------------
// Both backward contractions of a step in one launch:
//   problem 0   dQ partial[z] = G . T     A = dL/dF read K-major,  B = negatives read MN-major
//   problem 1   dT partial[z] = G^T . Q   A = dL/dF read MN-major, B = queries read MN-major
// Launched one after the other, each gave every CTA a single item, so the pipeline fill, the drain
// of the accumulator and the launch were exposed twice (11-18 us of 41-47 us at B = 4096,
// N = 16384, d = 256).  Here the items of both problems form one list that the CTAs take in
// strides, two items per CTA at the shapes above, and the second item's MMAs run under the first
// item's drain (the accumulators are used in turn, as in tc_gemm_kernel).  Plain stores of fp32
// tiles; warp roles, barriers and bounded waits as in tc_gemm_kernel.
// ------------------------------------------------------------------------------------------
struct DualProb {
    int M, N, kb_total, kb_per_split, tiles_m, tiles_n, items;
    float* C; int64_t ldc, split_stride;
    // K in segments of seg_kb slices: the B operand's K coordinate starts over with every segment, and an MN-major
    // A operand moves a_seg_x columns to the right per segment instead of going on downwards (its segments lie
    // side by side in memory).  One segment = a plain contraction.
    int seg_kb, a_seg_x;
    // fold > 0: output column c goes to column c % fold of slab c / fold (slabs fold_stride floats apart)
    int fold; int64_t fold_stride;
};

// PAIR: the A operand has two K segments that meet the same slices of the B operand (two-term splits of dL/dF-like
// coefficients against one [x1 | x2] operand).  A stage then holds both segments' A tiles beside the one B tile and both
// are multiplied into the accumulator, so a B slice is fetched once instead of once per segment (a third fewer operand
// bytes per flop); K runs over one segment's slices.  Three stages instead of four fit.
template <int BN, bool PAIR = false>
__global__ void __launch_bounds__(32 * (2 + TC_EPI_WARPS), 1) tc_gemm_dual_kernel(const __grid_constant__ CUtensorMap tmA0,
                                                                                    const __grid_constant__ CUtensorMap tmB0,
                                                                                    const __grid_constant__ CUtensorMap tmA1,
                                                                                    const __grid_constant__ CUtensorMap tmB1,
                                                                                    DualProb q0, DualProb q1, int32_t* status, int wait_limit) {
    constexpr uint32_t A_BYTES = PAIR ? 2 * TC_A_BYTES : TC_A_BYTES;      // A tile(s) of a stage; the B tile follows
    constexpr uint32_t STAGE_BYTES = tc_stage_bytes(BN) + (PAIR ? TC_A_BYTES : 0u);
    constexpr int STAGES = PAIR ? 3 : TC_STAGES;
    constexpr int NACC = 512 / BN;
    constexpr uint32_t TMEM_COLS = NACC * BN;
    constexpr int EW = TC_EPI_WARPS, EG = EW / 4;
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* base = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(base + (size_t)STAGES * STAGE_BYTES);
    uint64_t* empty = full + TC_RING_MAX;
    uint64_t* acc_full = empty + TC_RING_MAX;
    uint64_t* acc_empty = acc_full + NACC;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + NACC);
    volatile uint32_t* stop = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total = q0.items + q1.items;
    // item -> (problem, K split, first row, first column); column tile fastest inside a problem
    auto prob_of = [&](int item) { return item < q0.items ? 0 : 1; };
    auto item_of = [&](const DualProb& q, int local_item) {
        const int tn = local_item % q.tiles_n, r = local_item / q.tiles_n;
        return TcItem{r / q.tiles_m, (r % q.tiles_m) * TC_BM, tn * BN};
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < NACC; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EW); }
        *stop = 0;
        mbar_init_fence();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int ring = 0;
            for (int item = blockIdx.x; item < total && !*stop; item += gridDim.x) {
                const int which = prob_of(item);
                const DualProb q = which ? q1 : q0;
                const TcItem it = item_of(q, which ? item - q0.items : item);
                const CUtensorMap* ta = which ? &tmA1 : &tmA0;
                const CUtensorMap* tb = which ? &tmB1 : &tmB0;
                const int kb0 = it.z * q.kb_per_split, nkb = min(q.kb_per_split, q.kb_total - kb0);
                for (int kb = 0; kb < nkb; ++kb, ++ring) {
                    const int s = ring % STAGES;
                    if (!mbar_wait_idle(&empty[s], ((ring / STAGES) & 1) ^ 1, wait_limit)) { *stop = 1; set_status(status, KGE_ERR_TIMEOUT); break; }
                    unsigned char* sa = base + (size_t)s * STAGE_BYTES;
                    mbar_arrive_expect_tx(&full[s], STAGE_BYTES);
                    const int kblk = kb0 + kb, seg = PAIR ? 0 : kblk / q.seg_kb;
                    const int k0 = kblk * TC_BK, kseg = (kblk - seg * q.seg_kb) * TC_BK;
#pragma unroll
                    for (int half = 0; half < (PAIR ? 2 : 1); ++half) {       // PAIR: both segments' A tiles of this slice
                        unsigned char* da = sa + half * TC_A_BYTES;
                        if (which) {      // dL/dF with the contraction index as rows: two boxes of 64 output rows
#pragma unroll
                            for (int g = 0; g < TC_BM / 64; ++g)
                                tma_load_2d(da + g * TC_MN_GROUP_BYTES, ta, it.m0 + 64 * g + (PAIR ? half : seg) * q.a_seg_x, kseg, &full[s]);
                        } else {
                            tma_load_2d(da, ta, k0 + half * q.seg_kb * TC_BK, it.m0, &full[s]);
                        }
                    }
#pragma unroll
                    for (int g = 0; g < BN / 64; ++g) tma_load_2d(sa + A_BYTES + g * TC_MN_GROUP_BYTES, tb, it.n0 + 64 * g, kseg, &full[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_k = umma_idesc_bf16(TC_BM, BN, false, true), idesc_mn = umma_idesc_bf16(TC_BM, BN, true, true);
            int ring = 0;
            bool ok = true;
            for (int item = blockIdx.x, local = 0; item < total && ok && !*stop; item += gridDim.x, ++local) {
                const int which = prob_of(item);
                const DualProb q = which ? q1 : q0;
                const TcItem it = item_of(q, which ? item - q0.items : item);
                const int nkb = min(q.kb_per_split, q.kb_total - it.z * q.kb_per_split);
                const int buf = local % NACC;
                if (!mbar_wait_idle(&acc_empty[buf], ((local / NACC) & 1) ^ 1, wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)buf * BN;
                for (int kb = 0; kb < nkb; ++kb, ++ring) {
                    const int s = ring % STAGES;
                    if (!mbar_wait_idle(&full[s], (ring / STAGES) & 1, wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(base + (size_t)s * STAGE_BYTES);
#pragma unroll
                    for (int half = 0; half < (PAIR ? 2 : 1); ++half) {
#pragma unroll
                        for (int k = 0; k < TC_BK / 16; ++k) {
                            const uint32_t aa = sa + half * TC_A_BYTES;
                            const uint64_t ad = which ? umma_desc_mn_sw128(aa + k * 2048) : umma_desc_k_sw128(aa + k * 32);
                            const uint64_t bd = umma_desc_mn_sw128(sa + A_BYTES + k * 2048);
                            umma_bf16(tmem_acc, ad, bd, which ? idesc_mn : idesc_k, (kb | k | half) != 0);
                        }
                    }
                    umma_commit(&empty[s]);
                }
                umma_commit(&acc_full[buf]);           // also after a failed wait, so the epilogue warps wake up
            }
            if (!ok) { *stop = 1; set_status(status, KGE_ERR_TIMEOUT); }
        }
    } else {
        const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
        const int cgrp = (warp - 2) >> 2;              // which half of the tile's columns
        constexpr int COLS = BN / EG;
        float4* st = reinterpret_cast<float4*>(base + (size_t)STAGES * STAGE_BYTES + 256) + (size_t)(warp - 2) * (TC_STORE_STAGE_BYTES / 16);
        for (int item = blockIdx.x, local = 0; item < total; item += gridDim.x, ++local) {
            const int buf = local % NACC;
            const bool ok = mbar_wait_bounded(&acc_full[buf], (local / NACC) & 1, wait_limit);
            tc_fence_after();
            if (!ok || *stop) { if (lane == 0) { *stop = 1; set_status(status, KGE_ERR_TIMEOUT); } break; }
            const int which = prob_of(item);
            const DualProb q = which ? q1 : q0;
            const TcItem it = item_of(q, which ? item - q0.items : item);
            const int row = it.m0 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cgrp * COLS);
            float* const Cout = q.C + (int64_t)it.z * q.split_stride;
#pragma unroll 1
            for (int c0 = cgrp * COLS; c0 < (cgrp + 1) * COLS; c0 += 32) {
                float v[32];
                tmem_ld32(taddr + (uint32_t)(c0 - cgrp * COLS), v);
                const int ncol = it.n0 + c0;
                float* piece = Cout + ncol;                    // column ncol of row 0 of this item's slab
                if (q.fold > 0) piece += (int64_t)(ncol / q.fold) * (q.fold_stride - q.fold);   // (32-column pieces never straddle a fold)
                if (ncol + 32 <= q.N && (q.ldc & 3) == 0) {    // (warp-uniform) through shared memory: four rows' whole 128 bytes per store instruction
                    const int sw = lane & 7, row0 = row - lane;
#pragma unroll
                    for (int i = 0; i < 8; ++i) st[lane * 8 + (i ^ sw)] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int r = j * 4 + (lane >> 3), c = lane & 7;
                        const float4 val = st[r * 8 + (c ^ (r & 7))];
                        if (row0 + r < q.M) *reinterpret_cast<float4*>(piece + (int64_t)(row0 + r) * q.ldc + 4 * c) = val;
                    }
                    __syncwarp();
                } else if (row < q.M) {
                    float* dst = piece + (int64_t)row * q.ldc;
#pragma unroll
                    for (int i = 0; i < 32; ++i) if (ncol + i < q.N) dst[i] = v[i];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

// ------------------------------------------------------------------------------------------
// C[M, N] = A . B^T in fp32 accuracy from bf16 operands: both operands arrive as three-term splits x = x1 + x2 + x3 laid
// out side by side, [x1 | x2 | x3] with `tstride` columns per term (K rounded up to 64, padding zero), and the six
// products a_i b_j with i + j <= 4 are accumulated in fp32 (what is left out is below 2^-25 relative).  A stage holds
// one 64-wide K slice of all three terms of both operands (6 x 16 KB), so every slice is fetched once for the up to
// three products it takes part in: half the operand bytes of the same products run as one long K (each term's slice would
// be fetched once per product).  128 x 128 tiles, two stages, four accumulators in turn; warp roles, barriers and bounded
// waits as in tc_gemm_kernel; fp32 tiles leave through shared memory (see tc_epilogue).
// ------------------------------------------------------------------------------------------
struct TermsParams {
    int M, N, kslices, tstride;     // kslices = tstride / 64
    int tiles_m, tiles_n, items;    // column tile fastest
    float* C; int64_t ldc;
    int32_t* status; int wait_limit;
};
constexpr uint32_t TT_TERM_BYTES = 128 * TC_BK * 2;           // one term's 128 x 64 bf16 tile
constexpr uint32_t TT_STAGE_BYTES = 6 * TT_TERM_BYTES;
constexpr int TT_STAGES = 2;
constexpr size_t TT_SMEM = 1024 + (size_t)TT_STAGES * TT_STAGE_BYTES + 256 + (size_t)TC_EPI_WARPS * TC_STORE_STAGE_BYTES;

__global__ void __launch_bounds__(32 * (2 + TC_EPI_WARPS), 1) tc_gemm_terms_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                                     const __grid_constant__ CUtensorMap tmB, TermsParams p) {
    constexpr int BN = 128, NACC = 512 / BN;
    constexpr uint32_t TMEM_COLS = 512;
    extern __shared__ unsigned char tc_smem_raw[];
    unsigned char* base = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(base + (size_t)TT_STAGES * TT_STAGE_BYTES);
    uint64_t* empty = full + TT_STAGES;
    uint64_t* acc_full = empty + TT_STAGES;
    uint64_t* acc_empty = acc_full + NACC;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + NACC);
    volatile uint32_t* stop = tmem_slot + 1;
    float4* store_stage = reinterpret_cast<float4*>(base + (size_t)TT_STAGES * TT_STAGE_BYTES + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TT_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < NACC; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], TC_EPI_WARPS); }
        *stop = 0;
        mbar_init_fence();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int ring = 0;
            for (int item = blockIdx.x; item < p.items && !*stop; item += gridDim.x) {
                const int m0 = (item / p.tiles_n) * TC_BM, n0 = (item % p.tiles_n) * BN;
                for (int ks = 0; ks < p.kslices; ++ks, ++ring) {
                    const int s = ring % TT_STAGES;
                    if (!mbar_wait_idle(&empty[s], ((ring / TT_STAGES) & 1) ^ 1, p.wait_limit)) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); break; }
                    unsigned char* sa = base + (size_t)s * TT_STAGE_BYTES;
                    mbar_arrive_expect_tx(&full[s], TT_STAGE_BYTES);
#pragma unroll
                    for (int t = 0; t < 3; ++t) {
                        tma_load_2d(sa + t * TT_TERM_BYTES, &tmA, t * p.tstride + ks * TC_BK, m0, &full[s]);
                        tma_load_2d(sa + (3 + t) * TT_TERM_BYTES, &tmB, t * p.tstride + ks * TC_BK, n0, &full[s]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, BN, false, false);
            int ring = 0;
            bool ok = true;
            for (int item = blockIdx.x, local = 0; item < p.items && ok && !*stop; item += gridDim.x, ++local) {
                const int buf = local % NACC;
                if (!mbar_wait_idle(&acc_empty[buf], ((local / NACC) & 1) ^ 1, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)buf * BN;
                for (int ks = 0; ks < p.kslices; ++ks, ++ring) {
                    const int s = ring % TT_STAGES;
                    if (!mbar_wait_idle(&full[s], (ring / TT_STAGES) & 1, p.wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(base + (size_t)s * TT_STAGE_BYTES);
#pragma unroll
                    for (int ta = 0; ta < 3; ++ta) {
#pragma unroll
                        for (int tb = 0; tb < 3; ++tb) {
                            if (ta + tb > 2) continue;          // the six products that matter (terms counted from 0)
#pragma unroll
                            for (int k = 0; k < TC_BK / 16; ++k) {
                                const uint64_t ad = umma_desc_k_sw128(sa + ta * TT_TERM_BYTES + k * 32);
                                const uint64_t bd = umma_desc_k_sw128(sa + (3 + tb) * TT_TERM_BYTES + k * 32);
                                umma_bf16(tmem_acc, ad, bd, idesc, (ks | ta | tb | k) != 0);
                            }
                        }
                    }
                    umma_commit(&empty[s]);
                }
                umma_commit(&acc_full[buf]);           // also after a failed wait, so the epilogue warps wake up
            }
            if (!ok) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); }
        }
    } else {
        const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
        const int cgrp = (warp - 2) >> 2;              // which half of the tile's columns
        constexpr int COLS = BN / (TC_EPI_WARPS / 4);
        float4* st = store_stage + (size_t)(warp - 2) * (TC_STORE_STAGE_BYTES / 16);
        for (int item = blockIdx.x, local = 0; item < p.items; item += gridDim.x, ++local) {
            const int buf = local % NACC;
            const bool ok = mbar_wait_bounded(&acc_full[buf], (local / NACC) & 1, p.wait_limit);
            tc_fence_after();
            if (!ok || *stop) { if (lane == 0) { *stop = 1; set_status(p.status, KGE_ERR_TIMEOUT); } break; }
            const int m0 = (item / p.tiles_n) * TC_BM, n0 = (item % p.tiles_n) * BN;
            const int row0 = m0 + quarter * 32, row = row0 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cgrp * COLS);
#pragma unroll 1
            for (int c0 = cgrp * COLS; c0 < (cgrp + 1) * COLS; c0 += 32) {
                float v[32];
                tmem_ld32(taddr + (uint32_t)(c0 - cgrp * COLS), v);
                const int ncol = n0 + c0;
                if (ncol + 32 <= p.N && (p.ldc & 3) == 0) {      // (warp-uniform) four rows' whole 128 bytes per store instruction
                    const int sw = lane & 7;
#pragma unroll
                    for (int i = 0; i < 8; ++i) st[lane * 8 + (i ^ sw)] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int r = j * 4 + (lane >> 3), c = lane & 7;
                        const float4 val = st[r * 8 + (c ^ (r & 7))];
                        if (row0 + r < p.M) *reinterpret_cast<float4*>(p.C + (int64_t)(row0 + r) * p.ldc + ncol + 4 * c) = val;
                    }
                    __syncwarp();
                } else if (row < p.M) {
                    float* dst = p.C + (int64_t)row * p.ldc + ncol;
#pragma unroll
                    for (int i = 0; i < 32; ++i) if (ncol + i < p.N) dst[i] = v[i];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

}  // namespace

// Tensor map of a row-major bf16 matrix [rows, cols] with leading dimension ld (ld % 8 == 0,
// base 16-byte aligned) read in boxes of box_rows rows x 64 columns with the 128-byte swizzle
// (128 rows for a K-major operand tile, 64 for an MN-major one); what a box covers beyond the
// matrix reads as zero.
int tc_make_operand_map(kge_handle* h, void* map_out, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) { std::snprintf(h->cuda_err, sizeof(h->cuda_err), "cuTensorMapEncodeTiled is not available from this driver"); return KGE_ERR_CUDA; }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                          dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { std::snprintf(h->cuda_err, sizeof(h->cuda_err), "cuTensorMapEncodeTiled failed with code %d", (int)r); return KGE_ERR_CUDA; }
    return KGE_OK;
}

int tc_make_f32_tile_map(kge_handle* h, void* map_out, const void* base, int64_t rows, int64_t cols) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) { std::snprintf(h->cuda_err, sizeof(h->cuda_err), "cuTensorMapEncodeTiled is not available from this driver"); return KGE_ERR_CUDA; }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {32, 64};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base),
                          dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { std::snprintf(h->cuda_err, sizeof(h->cuda_err), "cuTensorMapEncodeTiled failed with code %d", (int)r); return KGE_ERR_CUDA; }
    return KGE_OK;
}

namespace {

// One warp per positive merges the per-piece statistics of its row (and the positive score,
// which the sampled softmax normalises over too) into the row's final (max, 1 / normaliser),
// the per-positive loss and dL/df+.
struct CombineParams {
    const float4* stat_part; int pieces; int B;
    const float* fpos;
    int loss; float gamma, ce_c, loss_scale;
    float2* row_stat; float *Lrow, *gpos;
};

__global__ void __launch_bounds__(256) stats_combine_kernel(CombineParams p) {
    const int b = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (b >= p.B) return;
    const float4* row = p.stat_part + (int64_t)b * p.pieces;
    const float fp = p.fpos[b];
    const bool ce = p.loss == KGE_LOSS_SAMPLED_SOFTMAX;
    // the pieces carry their maxima and exponent sums in base 2 (exponent times log2 e)
    float m = -INFINITY;
    for (int j = lane; j < p.pieces; j += 32) m = fmaxf(m, row[j].x);
    m = warp_max(m);
    if (ce) m = fmaxf(m, fp * kLog2e);
    float z = 0.f, l = 0.f;
    for (int j = lane; j < p.pieces; j += 32) {
        const float4 s = row[j];
        const float r = exp2f(s.x - m);    // a piece without valid columns has max = -inf: weight 0
        z += s.y * r; l += s.z * r;
    }
    z = warp_sum(z); l = warp_sum(l);
    if (lane != 0) return;
    if (ce) {
        const float epos = exp2f(fp * kLog2e - m);
        z += epos;
        p.Lrow[b] = -fp + (m + log2f(z)) * 0.6931471805599453f;
        p.gpos[b] = p.loss_scale * (epos / z - 1.f);
    } else {
        const float zp = -(p.gamma + fp), ep = expf(-fabsf(zp)), rp = 1.f / (1.f + ep);   // once per row: the exact forms
        const float sp = fmaxf(zp, 0.f) + log1pf(ep), sg = zp >= 0.f ? rp : ep * rp;
        p.Lrow[b] = sp + l / z;
        p.gpos[b] = -p.loss_scale * sg;
    }
    p.row_stat[b] = make_float2(m, 1.f / z);
}

// Norm expansion only: row sums and column sums of the written dL/dF from their pieces,
// added in ascending piece order.
__global__ void __launch_bounds__(256) grad_sums_kernel(const float* grow_part, int row_pieces, float* Grow, int B,
                                                        const float* gcol_part, int col_pieces, float* Gcol, int N) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < B) {
        float t = 0.f;
        for (int j = 0; j < row_pieces; ++j) t += grow_part[(int64_t)i * row_pieces + j];
        Grow[i] = t;
    } else if (i - B < N) {
        const int n = i - B;
        float t = 0.f;
        for (int j = 0; j < col_pieces; ++j) t += gcol_part[(int64_t)j * N + n];
        Gcol[n] = t;
    }
}

}  // namespace

namespace {
template <int EPI, int BN = 128, bool A_MN = false, bool B_MN = false>
cudaError_t launch_gemm_inst(const unsigned char* tmA, const unsigned char* tmB, const TcGemmParams& p, int num_sms, cudaStream_t s,
                             size_t extra_smem = 0) {
    constexpr size_t smem = tc_smem_bytes(BN);
    constexpr size_t extra_max = (EPI & 3) == EPI_TOPK ? (size_t)TC_BEAT_ROWS_MAX * 4
                               : ((EPI & 3) == EPI_GRAD ? (size_t)tc_epi_warps(EPI, BN) * TC_GRAD_STAGE_BYTES
                               : ((EPI & 3) == EPI_STORE ? (size_t)tc_epi_warps(EPI, BN) * TC_STORE_STAGE_BYTES : 0));
    if ((EPI & 3) == EPI_GRAD || (EPI & 3) == EPI_STORE) extra_smem = extra_max;
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        return cudaFuncSetAttribute(tc_gemm_kernel<EPI, BN, A_MN, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem + extra_max));
    });
    if (e != cudaSuccess) return e;
    tc_gemm_kernel<EPI, BN, A_MN, B_MN><<<std::min(p.items, num_sms), tc_threads(EPI, BN), smem + extra_smem, s>>>(
        *reinterpret_cast<const CUtensorMap*>(tmA), *reinterpret_cast<const CUtensorMap*>(tmB), p);
    return cudaSuccess;
}

// Scores Q . T^T with one of the fused loss epilogues, in tiles of BN columns.
template <int BN>
cudaError_t launch_fused_bn(int pass, bool l2, bool ce, kge_handle* h, const TcGemmParams& p, cudaStream_t s) {
    // the shared-exponential form of the log-sigmoid distance epilogues: temperature exactly 1, exp(gamma) finite
    if (l2 && !ce && p.adv_temp == 1.f && p.gamma <= 80.f) {
        if (pass == EPI_GRAD) return launch_gemm_inst<EPI_GRAD | EPI_L2 | EPI_A1, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        return launch_gemm_inst<EPI_STATS | EPI_L2 | EPI_A1, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
    }
    const int key = (pass == EPI_GRAD ? 4 : 0) | (l2 ? 2 : 0) | (ce ? 1 : 0);
    switch (key) {
        case 0: return launch_gemm_inst<EPI_STATS, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 1: return launch_gemm_inst<EPI_STATS | EPI_CE, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 2: return launch_gemm_inst<EPI_STATS | EPI_L2, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 3: return launch_gemm_inst<EPI_STATS | EPI_L2 | EPI_CE, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 4: return launch_gemm_inst<EPI_GRAD, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 5: return launch_gemm_inst<EPI_GRAD | EPI_CE, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        case 6: return launch_gemm_inst<EPI_GRAD | EPI_L2, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
        default: return launch_gemm_inst<EPI_GRAD | EPI_L2 | EPI_CE, BN>(h->tm_q, h->tm_t, p, h->num_sms, s);
    }
}
cudaError_t launch_fused(int pass, bool l2, bool ce, kge_handle* h, const TcGemmParams& p, cudaStream_t s) {
    return p.bn == 256 ? launch_fused_bn<256>(pass, l2, ce, h, p, s) : launch_fused_bn<128>(pass, l2, ce, h, p, s);
}
}  // namespace

// Forward of the tensor-core path without the B x N score block ever leaving the chip:
//   pass 1  scores -> per-piece statistics;  merge per row -> loss, dL/df+, (max, 1 / normaliser)
//   pass 2  scores again -> dL/dF as bf16, as it is and transposed, for the backward contractions
int launch_tc_forward(kge_handle* h, cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    TcGemmParams p{};
    p.M = c.batch; p.N = c.num_neg; p.K = c.dim;
    p.kb_per_split = (p.K + TC_BK - 1) / TC_BK; p.split_stride = 0;
    // 256-column tiles halve the operand bytes fetched per score (the row tile is shared by twice
    // the columns); narrow problems keep 128 so that the tiles still spread over the SMs
    p.bn = (p.N >= 1024 && (int64_t)((p.M + TC_BM - 1) / TC_BM) * ((p.N + 255) / 256) >= h->num_sms) ? 256 : TC_BN;
    p.tiles_m = (p.M + TC_BM - 1) / TC_BM; p.tiles_n = (p.N + p.bn - 1) / p.bn; p.items = p.tiles_m * p.tiles_n;
    p.row_pieces = TC_EPI_GROUPS * ((p.N + TC_BN - 1) / TC_BN);
    p.C = nullptr; p.ldc = 0;
    p.row_norm2 = w.qn2; p.col_norm2 = w.tn2;
    p.status = w.status; p.wait_limit = h->wait_limit;
    p.l2 = h->kind == KIND_L2; p.loss = c.loss;
    p.gamma = c.gamma; p.adv_temp = c.adv_temp; p.ce_c = c.ce_correction; p.loss_scale = c.loss_scale;
    p.stat_part = reinterpret_cast<float4*>(w.stat_part); p.row_stat = reinterpret_cast<const float2*>(w.row_stat);
    p.Gb = w.Gb; p.ldg = (c.num_neg + 7) / 8 * 8;
    p.grow_part = w.grow_part; p.gcol_part = w.gcol_part;
    const bool ce = c.loss == KGE_LOSS_SAMPLED_SOFTMAX;
    if (h->capture_scores) {
        // debug tap: this path never stores the score block, so an extra contraction writes it (fp32 [B, N]) with the
        // same mainloop and, for the norm expansion, the same score formula as the fused epilogues
        TcGemmParams cp = p;
        cp.bn = TC_BN; cp.tiles_n = (p.N + TC_BN - 1) / TC_BN; cp.items = cp.tiles_m * cp.tiles_n;
        cp.C = h->capture_scores; cp.ldc = p.N;
        if (p.l2) KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE | EPI_L2, 128>(h->tm_q, h->tm_t, cp, h->num_sms, s)));
        else KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE, 128>(h->tm_q, h->tm_t, cp, h->num_sms, s)));
        KGE_LAUNCH_CHECK(h);
    }
    stage_begin(h, ST_BLOCK, s);
    KGE_CUDA_CHECK(h, launch_fused(EPI_STATS, p.l2 != 0, ce, h, p, s));
    stage_end(h, ST_BLOCK, s);
    KGE_LAUNCH_CHECK(h);
    stage_begin(h, ST_LOSS, s);
    CombineParams cp{p.stat_part, p.row_pieces, p.M, w.fpos, c.loss, c.gamma, c.ce_correction, c.loss_scale,
                     reinterpret_cast<float2*>(w.row_stat), w.Lrow, w.gpos};
    stats_combine_kernel<<<(p.M * 32 + 255) / 256, 256, 0, s>>>(cp);
    KGE_LAUNCH_CHECK(h);
    KGE_CUDA_CHECK(h, launch_fused(EPI_GRAD, p.l2 != 0, ce, h, p, s));
    KGE_LAUNCH_CHECK(h);
    if (p.l2) {
        grad_sums_kernel<<<(p.M + p.N + 255) / 256, 256, 0, s>>>(w.grow_part, p.row_pieces, w.Grow, p.M,
                                                                 w.gcol_part, 4 * p.tiles_m, w.Gcol, p.N);
        KGE_LAUNCH_CHECK(h);
    }
    stage_end(h, ST_LOSS, s);
    return KGE_OK;
}

namespace {
// One backward contraction C[M, N] (+ K splits) with the tile width that fits the row width.
template <bool A_MN>
int launch_tc_bwd_gemm(kge_handle* h, const unsigned char* tmA, const unsigned char* tmB, int M, int N, int K, int split,
                       float* C, int64_t ldc, cudaStream_t s) {
    TcGemmParams p{};
    p.M = M; p.N = N; p.K = K;
    const int kb = (K + TC_BK - 1) / TC_BK;
    p.kb_per_split = (kb + split - 1) / split;
    p.C = C; p.ldc = ldc; p.split_stride = (int64_t)M * ldc;
    p.status = h->ws.status; p.wait_limit = h->wait_limit;
    p.bn = tc_backward_tile_cols(N);
    p.tiles_m = (M + TC_BM - 1) / TC_BM; p.tiles_n = (N + p.bn - 1) / p.bn;
    p.items = p.tiles_m * p.tiles_n * ((kb + p.kb_per_split - 1) / p.kb_per_split);
    if (p.bn == 256) KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE, 256, A_MN, true>(tmA, tmB, p, h->num_sms, s)));
    else KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE, 128, A_MN, true>(tmA, tmB, p, h->num_sms, s)));
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}
}  // namespace

namespace {
DualProb dual_prob(int M, int N, int K, int split, float* C, int64_t ldc, int bn) {
    DualProb q{};
    q.M = M; q.N = N;
    q.kb_total = (K + TC_BK - 1) / TC_BK;
    q.kb_per_split = (q.kb_total + split - 1) / split;
    q.tiles_m = (M + TC_BM - 1) / TC_BM; q.tiles_n = (N + bn - 1) / bn;
    q.items = q.tiles_m * q.tiles_n * ((q.kb_total + q.kb_per_split - 1) / q.kb_per_split);
    q.C = C; q.ldc = ldc; q.split_stride = (int64_t)M * ldc;
    q.seg_kb = q.kb_total; q.a_seg_x = 0; q.fold = 0; q.fold_stride = 0;
    return q;
}
template <int BN, bool PAIR = false>
cudaError_t launch_gemm_dual(kge_handle* h, const unsigned char* tmA0, const unsigned char* tmB0, const unsigned char* tmA1,
                             const unsigned char* tmB1, const DualProb& q0, const DualProb& q1, cudaStream_t s) {
    constexpr size_t smem = (PAIR ? 1024 + (size_t)3 * (tc_stage_bytes(BN) + TC_A_BYTES) + 256 : tc_smem_bytes(BN)) +
                            (size_t)TC_EPI_WARPS * TC_STORE_STAGE_BYTES;      // + the epilogue warps' store staging
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        return cudaFuncSetAttribute(tc_gemm_dual_kernel<BN, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    });
    if (e != cudaSuccess) return e;
    // as few CTAs as give the same number of rounds: SMs left over serve the id sort that runs beside this launch
    const int total = q0.items + q1.items;
    const int rounds = (total + h->num_sms - 1) / h->num_sms;
    const int grid = (total + rounds - 1) / rounds;
    tc_gemm_dual_kernel<BN, PAIR><<<grid, 32 * (2 + TC_EPI_WARPS), smem, s>>>(
        *reinterpret_cast<const CUtensorMap*>(tmA0), *reinterpret_cast<const CUtensorMap*>(tmB0),
        *reinterpret_cast<const CUtensorMap*>(tmA1), *reinterpret_cast<const CUtensorMap*>(tmB1), q0, q1, h->ws.status, h->wait_limit);
    return cudaSuccess;
}
}  // namespace

// Plain contractions for the feature-projection encoder, on the same kernel.
//   C[M, N] = A[M, K] . B[N, K]^T   (both operands K-major: tensor maps with 128-row boxes)
int launch_tc_gemm_nt(kge_handle* h, const unsigned char* tmA, const unsigned char* tmB, int M, int N, int K, float* C, int64_t ldc,
                      cudaStream_t s) {
    TcGemmParams p{};
    p.M = M; p.N = N; p.K = K;
    p.kb_per_split = (K + TC_BK - 1) / TC_BK;
    p.C = C; p.ldc = ldc; p.split_stride = 0;
    p.status = h->ws.status; p.wait_limit = h->wait_limit;
    // 256-column tiles halve the operand bytes fetched per output once there are enough of them for every SM
    p.bn = (N >= 1024 && (int64_t)((M + TC_BM - 1) / TC_BM) * ((N + 255) / 256) >= h->num_sms) ? 256 : TC_BN;
    p.tiles_m = (M + TC_BM - 1) / TC_BM; p.tiles_n = (N + p.bn - 1) / p.bn; p.items = p.tiles_m * p.tiles_n;
    if (p.bn == 256) KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE, 256>(tmA, tmB, p, h->num_sms, s)));
    else KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_STORE, 128>(tmA, tmB, p, h->num_sms, s)));
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}
//   C[M, N] = A . B^T with fp32 accuracy from three-term bf16 splits [x1 | x2 | x3] of both operands (`tstride` columns per
//   term, a multiple of 64 with zero padding; tensor maps with 128-row boxes over [rows, 3 tstride])
int launch_tc_gemm_terms(kge_handle* h, const unsigned char* tmA, const unsigned char* tmB, int M, int N, int tstride, float* C,
                         int64_t ldc, cudaStream_t s) {
    TermsParams p{};
    p.M = M; p.N = N; p.tstride = tstride; p.kslices = tstride / TC_BK;
    p.tiles_m = (M + TC_BM - 1) / TC_BM; p.tiles_n = (N + 127) / 128; p.items = p.tiles_m * p.tiles_n;
    p.C = C; p.ldc = ldc; p.status = h->ws.status; p.wait_limit = h->wait_limit;
    static DeviceOnce configured;
    KGE_CUDA_CHECK(h, once_per_device(configured, [] {
        return cudaFuncSetAttribute(tc_gemm_terms_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TT_SMEM);
    }));
    tc_gemm_terms_kernel<<<std::min(p.items, h->num_sms), 32 * (2 + TC_EPI_WARPS), TT_SMEM, s>>>(
        *reinterpret_cast<const CUtensorMap*>(tmA), *reinterpret_cast<const CUtensorMap*>(tmB), p);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}
//   C[split][M, N] = A[K, M]^T . B[K, N] over K slices of each split (both operands MN-major: 64-row boxes)
int launch_tc_gemm_tn(kge_handle* h, const unsigned char* tmA64, const unsigned char* tmB64, int M, int N, int K, int split, float* C,
                      int64_t ldc, cudaStream_t s) {
    return launch_tc_bwd_gemm<true>(h, tmA64, tmB64, M, N, K, split, C, ldc, s);
}

bool tc_negatives_direct(const kge_handle* h) {
    // (with the regulariser on, the chain kernel still has a term to add to every negative's row)
    return h->cfg.prec == KGE_PREC_BF16_TC && h->kind == KIND_DOT && h->split_t == 1 && !(h->cfg.reg_lambda > 0.f);
}

// Columns per tile of a backward contraction whose output rows are `cols` wide.
int tc_backward_tile_cols(int cols) { return cols > 128 ? 256 : 128; }

// Column pieces per 128-wide tile for which the fused forward keeps separate statistics.
int tc_pieces_per_tile() { return TC_EPI_GROUPS; }

// The two backward contractions on tensor cores, from the bf16 dL/dF the forward left behind.
// No operand is transposed in memory: an operand whose contraction index is its row index is
// read MN-major.
//   dQ partial[split] = G . T      A = Gb [B, N] (K-major),          B operand = Tb [N, d] (MN-major)
//   dT partial[split] = G^T . Q    A = Gb [B, N] read MN-major,      B operand = Qb [B, d] (MN-major)
// The K splits land in the same partial buffers the CUDA-core path uses and are added in
// ascending order by the chain kernel.
int launch_tc_backward(kge_handle* h, cudaStream_t s, cudaStream_t side) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg, d = c.dim;
    (void)side;
    // one split and no correction term: the negatives' rows are final, so they go where the update reads them
    float* dT_out = tc_negatives_direct(h) ? w.grad_ent + (size_t)2 * B * d : w.dTpart;
    const int bn = tc_backward_tile_cols(d);
    const DualProb q0 = dual_prob(B, d, N, h->split_q, w.dQpart, d, bn), q1 = dual_prob(N, d, B, h->split_t, dT_out, d, bn);
    stage_begin(h, ST_ACCUM_Q, s);        // (both contractions: the profile reports them as one stage)
    KGE_CUDA_CHECK(h, bn == 256 ? launch_gemm_dual<256>(h, h->tm_g, h->tm_t64, h->tm_g64, h->tm_q64, q0, q1, s)
                                : launch_gemm_dual<128>(h, h->tm_g, h->tm_t64, h->tm_g64, h->tm_q64, q0, q1, s));
    stage_end(h, ST_ACCUM_Q, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

// TransH on the fp32 path: the two contractions of the backward whose coefficient is one number per pair,
//   dW_b += sum_n c_bn t_n      and      dT_n += sum_b c_bn w_b,
// from bf16 two-term splits x = x1 + x2 of all three operands.  With the splits side by side, [c1 | c2] over K and
// [x1 | x2] over the output columns, one pass forms c1 x1 + c2 x1 in the left half of a tile and c1 x2 + c2 x2 in
// the right half: all four products, accumulated in fp32; the halves (and the K splits) land in slabs of their own
// behind the CUDA-core kernels' slabs and the chain kernel adds them in order.
int th_contract_slabs(const kge_handle* h) { return h->th_tc ? 2 * h->th_gsplit : 0; }

int launch_th_contract_gemm(kge_handle* h, cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg, d = c.dim;
    const int Np = (N + 63) / 64 * 64, Bp = (B + 63) / 64 * 64;
    const int bn = tc_backward_tile_cols(2 * d);
    // (K runs over one segment: both segments' tiles of c travel in one stage, see tc_gemm_dual_kernel<BN, PAIR>)
    DualProb q0 = dual_prob(B, 2 * d, Np, h->th_gsplit, w.dWpart + (size_t)h->split_q * B * d, d, bn);
    DualProb q1 = dual_prob(N, 2 * d, Bp, h->th_gsplit, w.dTpart + (size_t)h->split_t * N * d, d, bn);
    q0.seg_kb = Np / TC_BK; q0.a_seg_x = 0;
    q1.seg_kb = Bp / TC_BK; q1.a_seg_x = Np;
    q0.fold = q1.fold = d;
    q0.fold_stride = (int64_t)B * d; q0.split_stride = 2 * q0.fold_stride;
    q1.fold_stride = (int64_t)N * d; q1.split_stride = 2 * q1.fold_stride;
    KGE_CUDA_CHECK(h, bn == 256 ? (launch_gemm_dual<256, true>(h, h->tm_cs, h->tm_ts64, h->tm_cs64, h->tm_ws64, q0, q1, s))
                                : (launch_gemm_dual<128, true>(h, h->tm_cs, h->tm_ts64, h->tm_cs64, h->tm_ws64, q0, q1, s)));
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}


namespace {
__global__ void __launch_bounds__(256) cast_bf16_kernel(const float4* src, uint2* dst, int64_t n4) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = src[i];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        dst[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
}
}  // namespace

// bf16 copy of `count` floats (count % 4 == 0, both 16-byte aligned).
int launch_cast_bf16(kge_handle* h, const float* src, uint16_t* dst, int64_t count, cudaStream_t s) {
    const int64_t n4 = count / 4;
    const int grid = (int)std::min<int64_t>((n4 + 255) / 256, (int64_t)h->num_sms * 16);
    cast_bf16_kernel<<<std::max(grid, 1), 256, 0, s>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(dst), n4);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

// One chunk of full-entity scoring on tensor cores: the bf16 query vectors against the bf16
// rows [e_lo, e_hi) of the entity table, survivors appended to the candidate lists.
int launch_tc_infer_chunk(kge_handle* h, int nq, int64_t e_lo, int64_t e_hi, const int32_t* true_tails, int64_t id_base, cudaStream_t s) {
    const Workspace& w = h->ws;
    TcGemmParams p{};
    p.M = nq; p.N = (int)(e_hi - e_lo); p.K = h->cfg.dim;
    p.kb_per_split = (p.K + TC_BK - 1) / TC_BK;
    p.bn = 256;      // a row tile of queries is shared by 256 entities
    p.tiles_m = (p.M + TC_BM - 1) / TC_BM; p.tiles_n = (p.N + p.bn - 1) / p.bn;
    if ((int64_t)p.tiles_m * p.tiles_n > 0x7fffffff) return KGE_ERR_BAD_ARG;
    p.items = p.tiles_m * p.tiles_n;
    p.status = w.status; p.wait_limit = h->wait_limit;
    p.m_fastest = 1; p.n_base = e_lo; p.id_base = id_base;
    p.thr = w.thr; p.thr_id = w.thr_id; p.ftrue = w.iftrue; p.tt = true_tails;
    p.cand_cnt = w.cand_cnt; p.beat_tmp = w.beat_tmp; p.cand_score = w.cand_score; p.cand_id = w.cand_id;
    p.cand_cap = kCandCap; p.overflow = w.status + 1;
    p.beat_rows = std::min(nq, TC_BEAT_ROWS_MAX);   // the other rows count with global atomics
    p.resident_b = p.kb_per_split <= 2 ? 1 : 0;     // the column tile's two slices fit beside an eight-stage ring of row-tile slices
    // (the table's tensor map covers all rows; the kernel offsets its row coordinate by n_base)
    KGE_CUDA_CHECK(h, (launch_gemm_inst<EPI_TOPK, 256>(h->tm_iq, h->tm_eb, p, h->num_sms, s, (size_t)p.beat_rows * 4)));
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
