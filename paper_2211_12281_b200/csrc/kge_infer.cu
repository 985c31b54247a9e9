// Full-entity inference (Section 3.1 "Inference"): every query is scored against every
// entity; per query the k best tails under (score descending, id ascending) and the rank
// of the true tail.  The entity table is streamed once, in chunks that grow geometrically;
// inside a chunk a pair survives only if it beats the query's current k-th best, survivors
// are appended to a per-query candidate list, and a selection step between chunks merges
// them into the running top-k and tightens the threshold (the single-device analogue of the
// per-worker top-K followed by a final top-K over the gathered candidates).
//
// fp32 arithmetic here is "canonical": per pair one accumulator, embedding index ascending,
// rounding exactly where written (intrinsics keep the compiler from fusing anything else),
// so that ties and near-ties order the same way on any implementation of the same recipe.
#include <algorithm>
#include <climits>
#include <cmath>
#include <vector>

#include <cuda_bf16.h>

#include <cuda.h>

#include "kge_common.cuh"

namespace kge {

namespace {

struct InferParams {
    int nq, k, d, d4, score, kind;
    int64_t E, R;
    const float *ent, *rel, *relw;
    const int32_t *qh, *qr, *tt;   // tt may be NULL
    int64_t e_lo, e_hi;            // entity range of this launch
    int q_tiles;
    int wait_limit;                // tries of a bounded barrier wait
    // sharded inference (Section 4 "Inference"): the bound table is the shard [id_base, id_base + E) of a larger one;
    // query vectors and true-tail scores come from outside (they need rows of other shards), ids are global
    int64_t id_base;
    const float* ext_q;            // [nq, d] finished query vectors, or NULL: build them from qh, qr
    const float* ext_ftrue;        // [nq] scores of the true tails, or NULL: score them here
    int raw_beat;                  // out_ranks receives the shard's count of entities ordered before the true tail, not 1 + count
    Workspace w;
};

// One canonical accumulation step over the 4 floats of a slice.
template <int KIND>
__device__ __forceinline__ void canon_update(float& acc, float4 q, float4 t) {
    if (KIND == KIND_DOT) {
        acc = __fmaf_rn(q.x, t.x, acc); acc = __fmaf_rn(q.y, t.y, acc);
        acc = __fmaf_rn(q.z, t.z, acc); acc = __fmaf_rn(q.w, t.w, acc);
    } else if (KIND == KIND_L1) {
        acc = __fadd_rn(acc, fabsf(__fsub_rn(q.x, t.x))); acc = __fadd_rn(acc, fabsf(__fsub_rn(q.y, t.y)));
        acc = __fadd_rn(acc, fabsf(__fsub_rn(q.z, t.z))); acc = __fadd_rn(acc, fabsf(__fsub_rn(q.w, t.w)));
    } else if (KIND == KIND_L2) {
        float x;
        x = __fsub_rn(q.x, t.x); acc = __fmaf_rn(x, x, acc); x = __fsub_rn(q.y, t.y); acc = __fmaf_rn(x, x, acc);
        x = __fsub_rn(q.z, t.z); acc = __fmaf_rn(x, x, acc); x = __fsub_rn(q.w, t.w); acc = __fmaf_rn(x, x, acc);
    } else {  // KIND_CL1
        float xr = __fsub_rn(q.x, t.x), xi = __fsub_rn(q.y, t.y);
        acc = __fadd_rn(acc, __fsqrt_rn(__fmaf_rn(xr, xr, __fmul_rn(xi, xi))));
        xr = __fsub_rn(q.z, t.z); xi = __fsub_rn(q.w, t.w);
        acc = __fadd_rn(acc, __fsqrt_rn(__fmaf_rn(xr, xr, __fmul_rn(xi, xi))));
    }
}

__device__ __forceinline__ float4 canon_th_x(float u, float4 w, float4 q, float4 t) {
    return make_float4(__fmaf_rn(u, w.x, __fsub_rn(q.x, t.x)), __fmaf_rn(u, w.y, __fsub_rn(q.y, t.y)),
                       __fmaf_rn(u, w.z, __fsub_rn(q.z, t.z)), __fmaf_rn(u, w.w, __fsub_rn(q.w, t.w)));
}
__device__ __forceinline__ void canon_th_acc(int kind, float& acc, float4 x) {
    if (kind == KIND_TH_L1) {
        acc = __fadd_rn(acc, fabsf(x.x)); acc = __fadd_rn(acc, fabsf(x.y));
        acc = __fadd_rn(acc, fabsf(x.z)); acc = __fadd_rn(acc, fabsf(x.w));
    } else {
        acc = __fmaf_rn(x.x, x.x, acc); acc = __fmaf_rn(x.y, x.y, acc);
        acc = __fmaf_rn(x.z, x.z, acc); acc = __fmaf_rn(x.w, x.w, acc);
    }
}
__device__ __forceinline__ float canon_finish(int kind, float acc) {
    if (kind == KIND_DOT) return acc;
    if (kind == KIND_L2 || kind == KIND_TH_L2) return -__fsqrt_rn(acc);
    return -acc;
}

__device__ __forceinline__ bool ordered_before(float fa, int32_t ia, float fb, int32_t ib) {
    return fa > fb || (fa == fb && ia < ib);
}

// ------------------------------------------------------------------------------------------
// query set-up: one thread per query builds q (and the TransH unit normal) sequentially,
// scores the true tail, and resets the query's running state.
// ------------------------------------------------------------------------------------------
// TransH: the unit normal of relation rid into wh, sequentially.
__device__ __forceinline__ void unit_normal_seq(const InferParams& p, int64_t rid, float* wh) {
    const float* w = p.relw + rid * p.d;
    float s = 0.f;
    for (int k = 0; k < p.d; ++k) s = __fmaf_rn(w[k], w[k], s);
    const float den = fmaxf(__fsqrt_rn(s), 1e-12f);
    for (int k = 0; k < p.d; ++k) wh[k] = __fdiv_rn(w[k], den);
}

// Query vector of (head row h, relation rid) into qv (and the TransH unit normal into wh), sequentially.
__device__ __forceinline__ void build_query_seq(const InferParams& p, const float* h, int64_t rid, float* qv, float* wh) {
    const int d = p.d;
    if (p.score == KGE_TRANSE) {
        const float* r = p.rel + rid * d;
        for (int k = 0; k < d; ++k) qv[k] = __fadd_rn(h[k], r[k]);
    } else if (p.score == KGE_DISTMULT) {
        const float* r = p.rel + rid * d;
        for (int k = 0; k < d; ++k) qv[k] = __fmul_rn(r[k], h[k]);
    } else if (p.score == KGE_COMPLEX) {
        const float* r = p.rel + rid * d;
        for (int k = 0; k < d; k += 2) {
            qv[k] = __fmaf_rn(r[k], h[k], -__fmul_rn(r[k + 1], h[k + 1]));
            qv[k + 1] = __fmaf_rn(r[k], h[k + 1], __fmul_rn(r[k + 1], h[k]));
        }
    } else if (p.score == KGE_ROTATE) {
        const float* th = p.rel + rid * (d / 2);
        for (int k = 0; k < d; k += 2) {
            const float cs = cosf(th[k / 2]), sn = sinf(th[k / 2]);
            qv[k] = __fmaf_rn(h[k], cs, -__fmul_rn(h[k + 1], sn));
            qv[k + 1] = __fmaf_rn(h[k], sn, __fmul_rn(h[k + 1], cs));
        }
    } else {  // TransH
        const float* r = p.rel + rid * d;
        unit_normal_seq(p, rid, wh);
        float a = 0.f;
        for (int k = 0; k < d; ++k) a = __fmaf_rn(wh[k], h[k], a);
        for (int k = 0; k < d; ++k) qv[k] = __fadd_rn(__fmaf_rn(-a, wh[k], h[k]), r[k]);
    }
}

// Canonical score of (query vector qv, unit normal wh, tail row t).
__device__ __forceinline__ float score_seq(const InferParams& p, const float* qv, const float* wh, const float* t) {
    const int d = p.d;
    {
        float acc = 0.f;
        if (p.score == KGE_TRANSH) {
            float u = 0.f;
            for (int k = 0; k < d; ++k) u = __fmaf_rn(wh[k], t[k], u);
            for (int k = 0; k < d; k += 4)
                canon_th_acc(p.kind, acc, canon_th_x(u, *reinterpret_cast<const float4*>(wh + k),
                                                     *reinterpret_cast<const float4*>(qv + k),
                                                     *reinterpret_cast<const float4*>(t + k)));
        } else {
            for (int k = 0; k < d; k += 4) {
                const float4 q4 = *reinterpret_cast<const float4*>(qv + k);
                const float4 t4 = *reinterpret_cast<const float4*>(t + k);
                if (p.kind == KIND_DOT) canon_update<KIND_DOT>(acc, q4, t4);
                else if (p.kind == KIND_L1) canon_update<KIND_L1>(acc, q4, t4);
                else if (p.kind == KIND_L2) canon_update<KIND_L2>(acc, q4, t4);
                else canon_update<KIND_CL1>(acc, q4, t4);
            }
        }
        return canon_finish(p.kind, acc);
    }
}

__global__ void query_setup_kernel(InferParams p) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.nq) return;
    const int d = p.d;
    const int64_t rid = checked_id(p.qr[q], p.R, p.w.status);
    float* qv = p.w.iq + (int64_t)q * d;
    float* wh = p.score == KGE_TRANSH ? p.w.iwhat + (int64_t)q * d : nullptr;
    if (p.ext_q) {   // sharded: the query vector was built by the shard that holds the head
        for (int k = 0; k < d; ++k) qv[k] = p.ext_q[(int64_t)q * d + k];
        if (wh) unit_normal_seq(p, rid, wh);
    } else {
        build_query_seq(p, p.ent + checked_id(p.qh[q], p.E, p.w.status) * d, rid, qv, wh);
    }
    if (p.ext_ftrue) p.w.iftrue[q] = p.ext_ftrue[q];
    else if (p.tt) p.w.iftrue[q] = score_seq(p, qv, wh, p.ent + checked_id(p.tt[q], p.E, p.w.status) * d);
    for (int j = 0; j < p.k; ++j) {
        p.w.top_score[(int64_t)q * p.k + j] = -INFINITY;
        p.w.top_id[(int64_t)q * p.k + j] = INT_MAX;
    }
    p.w.thr[q] = -INFINITY; p.w.thr_id[q] = INT_MAX;
    p.w.cand_cnt[q] = 0; p.w.beat_tmp[q] = 0; p.w.beat[q] = 0;
}

constexpr int IQ = 64, IE = 64, IKC = 32, ILD = IKC + 4;

// Largest float below x (x finite).
__device__ __forceinline__ float float_below(float x) {
    if (x == 0.f) return __uint_as_float(0x80000001u);
    const uint32_t b = __float_as_uint(x);
    return __uint_as_float(x > 0.f ? b - 1u : b + 1u);
}

// Epilogue of a 64 x 64 score tile: rank counting against the true tail, threshold filter into the
// candidate lists.  Thread (tx, ty) holds the pairs (q0 + ty + 16 i, e0 + tx + 16 j).
// The tile's 64 entity ids are consecutive.  If the reference id (the true tail, or the id of the
// current k-th best) is not among them, "ordered before (f0, id0)" is the same plain comparison
// for the whole row of the tile: f >= f0 when the tile lies below id0, f > f0 when above, and
// f >= f0 is f > (largest float below f0).  So the common case costs one compare per pair and
// test; a row whose reference id falls inside the tile, a ragged last tile and non-finite
// reference scores take the element-by-element form.
//
// `cuts` (optional, shared memory, one entry per query row of the tile): the two comparison values of a row in the
// plain case, worked out once per row by score_tile_row_cuts while the tile's rows are still on their way, so that
// the sixteen threads of a row do not each load the row's state and form them again.
__device__ __forceinline__ void score_tile_row_cuts(const InferParams& p, int q0, int64_t e0, int row, float4* cuts) {
    const int64_t g0 = e0 + p.id_base;
    const int q = q0 + row;
    float4 c = make_float4(0.f, INFINITY, 0.f, 0.f);     // (x: candidate cut, y: rank cut, z: 1 = plain case)
    if (q < p.nq && e0 + IE <= p.e_hi) {
        const float thr = p.w.thr[q]; const int32_t thr_id = p.w.thr_id[q];
        float ft = 0.f; int32_t tt = -1;
        if (p.tt) { ft = p.w.iftrue[q]; tt = p.tt[q]; }
        const bool thr_out = thr_id < g0 || thr_id >= g0 + IE, tt_out = !p.tt || tt < g0 || tt >= g0 + IE;
        if (thr_out && tt_out && fabsf(thr) < INFINITY && fabsf(ft) < INFINITY) {
            c.x = thr_id >= g0 + IE ? float_below(thr) : thr;
            c.y = !p.tt ? INFINITY : (tt >= g0 + IE ? float_below(ft) : ft);     // without true tails nothing is counted
            c.z = 1.f;
        }
    }
    cuts[row] = c;
}

template <int KIND>
__device__ __forceinline__ void score_tile_epilogue(const InferParams& p, const float (&acc)[4][4], int q0, int64_t e0, int tx, int ty,
                                                    const float4* cuts = nullptr) {
    const int64_t g0 = e0 + p.id_base;                  // the id the caller knows the tile's first entity by
    const bool whole = e0 + IE <= p.e_hi;
    int beat_all = 0;                                   // four rows' counts, one byte each (at most 4 per thread, 64 per row)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int q = q0 + ty + 16 * i;
        const bool qin = q < p.nq;
        if (cuts) {
            const float4 c = cuts[ty + 16 * i];
            if (c.z != 0.f) {
                int beat = 0;
                float f[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { f[j] = canon_finish(KIND, acc[i][j]); beat += f[j] > c.y ? 1 : 0; }
                if (fmaxf(fmaxf(f[0], f[1]), fmaxf(f[2], f[3])) > c.x) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (f[j] > c.x) {
                            const int slot = atomicAdd(&p.w.cand_cnt[q], 1);
                            if (slot < kCandCap) {
                                p.w.cand_score[(int64_t)q * kCandCap + slot] = f[j];
                                p.w.cand_id[(int64_t)q * kCandCap + slot] = (int32_t)(g0 + tx + 16 * j);
                            } else {
                                p.w.status[1] = 1;
                            }
                        }
                }
                beat_all |= beat << (8 * i);
                continue;
            }
        }
        float thr = 0.f, ft = 0.f; int32_t thr_id = 0, tt = 0;
        if (qin) {
            thr = p.w.thr[q]; thr_id = p.w.thr_id[q];
            if (p.tt) { ft = p.w.iftrue[q]; tt = p.tt[q]; }
        }
        auto append = [&](float f, int32_t ge) {
            const int slot = atomicAdd(&p.w.cand_cnt[q], 1);
            if (slot < kCandCap) {
                p.w.cand_score[(int64_t)q * kCandCap + slot] = f;
                p.w.cand_id[(int64_t)q * kCandCap + slot] = ge;
            } else {
                p.w.status[1] = 1;   // this chunk overflowed a list: the host redoes it in small pieces
            }
        };
        const bool thr_out = thr_id < g0 || thr_id >= g0 + IE, tt_out = tt < g0 || tt >= g0 + IE;
        const bool plain = whole && qin && thr_out && tt_out && fabsf(thr) < INFINITY && fabsf(ft) < INFINITY;
        int beat = 0;
        if (plain) {
            const float thr_c = thr_id >= g0 + IE ? float_below(thr) : thr;
            const float ft_c = tt >= g0 + IE ? float_below(ft) : ft;
            float f[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { f[j] = canon_finish(KIND, acc[i][j]); beat += f[j] > ft_c ? 1 : 0; }
            // candidates are rare once the threshold has tightened: one test of the largest of the four
            // instead of four divergent branches
            if (fmaxf(fmaxf(f[0], f[1]), fmaxf(f[2], f[3])) > thr_c) {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (f[j] > thr_c) append(f[j], (int32_t)(g0 + tx + 16 * j));
            }
            if (!p.tt) beat = 0;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t e = e0 + tx + 16 * j;
                if (!qin || e >= p.e_hi) continue;
                const float f = canon_finish(KIND, acc[i][j]);
                const int32_t ge = (int32_t)(e + p.id_base);
                if (p.tt && ordered_before(f, ge, ft, tt)) ++beat;
                if (ordered_before(f, ge, thr, thr_id)) append(f, ge);
            }
        }
        beat_all |= beat << (8 * i);
    }
    // the 16 lanes sharing a query row are contiguous: one atomic per row and tile
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) beat_all += __shfl_xor_sync(0xffffffffu, beat_all, o);
    if (tx == 0 && beat_all != 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int beat = (beat_all >> (8 * i)) & 0xff;
            if (beat > 0) atomicAdd(&p.w.beat_tmp[q0 + ty + 16 * i], beat);
        }
    }
}

// ------------------------------------------------------------------------------------------
// score tile: 64 queries x 64 entities per CTA, 4 x 4 pairs per thread.  Consecutive CTAs
// walk the query tiles of one entity tile, so an entity tile is fetched from HBM once and
// served to the other query tiles by L2.
// ------------------------------------------------------------------------------------------
template <int KIND>
__global__ void __launch_bounds__(256) score_tile_kernel(InferParams p) {
    constexpr bool TH = KIND == KIND_TH_L1 || KIND == KIND_TH_L2;
    __shared__ __align__(16) float Qs[IQ * ILD];
    __shared__ __align__(16) float Ts[IE * ILD];
    __shared__ __align__(16) float Ws[TH ? IQ * ILD : 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int qt = blockIdx.x % p.q_tiles;
    const int64_t et = blockIdx.x / p.q_tiles;
    const int q0 = qt * IQ;
    const int64_t e0 = p.e_lo + et * IE;
    const int d4 = p.d4;
    const float4* Qg = reinterpret_cast<const float4*>(p.w.iq);
    const float4* Wg = reinterpret_cast<const float4*>(p.w.iwhat);
    const float4* Tg = reinterpret_cast<const float4*>(p.ent);

    __shared__ float4 cuts[IQ];
    if (tid >= 256 - IQ) score_tile_row_cuts(p, q0, e0, tid - (256 - IQ), cuts);     // (read after the barriers of the loop below)
    float acc[4][4], u[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; u[i][j] = 0.f; }
    const int npass = TH ? 2 : 1;
    for (int pass = 0; pass < npass; ++pass) {
        const bool upass = TH && pass == 0;
        for (int k0 = 0; k0 < p.d; k0 += IKC) {
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int idx = tid + 256 * it, row = idx >> 3, c4 = idx & 7;
                const int gc = (k0 >> 2) + c4;
                const bool kin = gc < d4;
                float4 qv = make_float4(0.f, 0.f, 0.f, 0.f), tv = qv, wv = qv;
                if (kin && q0 + row < p.nq) {
                    qv = Qg[(int64_t)(q0 + row) * d4 + gc];
                    if (TH) wv = Wg[(int64_t)(q0 + row) * d4 + gc];
                }
                if (kin && e0 + row < p.e_hi) tv = Tg[(e0 + row) * d4 + gc];
                *reinterpret_cast<float4*>(&Qs[row * ILD + c4 * 4]) = qv;
                *reinterpret_cast<float4*>(&Ts[row * ILD + c4 * 4]) = tv;
                if (TH) *reinterpret_cast<float4*>(&Ws[row * ILD + c4 * 4]) = wv;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < IKC; kk += 4) {
                float4 qv[4], tv[4], wv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    qv[i] = *reinterpret_cast<const float4*>(&Qs[(ty + 16 * i) * ILD + kk]);
                    tv[i] = *reinterpret_cast<const float4*>(&Ts[(tx + 16 * i) * ILD + kk]);
                    if (TH) wv[i] = *reinterpret_cast<const float4*>(&Ws[(ty + 16 * i) * ILD + kk]);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (!TH) {
                            canon_update<TH ? KIND_L1 : KIND>(acc[i][j], qv[i], tv[j]);
                        } else if (upass) {
                            u[i][j] = __fmaf_rn(wv[i].x, tv[j].x, u[i][j]); u[i][j] = __fmaf_rn(wv[i].y, tv[j].y, u[i][j]);
                            u[i][j] = __fmaf_rn(wv[i].z, tv[j].z, u[i][j]); u[i][j] = __fmaf_rn(wv[i].w, tv[j].w, u[i][j]);
                        } else {
                            canon_th_acc(KIND, acc[i][j], canon_th_x(u[i][j], wv[i], qv[i], tv[j]));
                        }
                    }
            }
            __syncthreads();
        }
    }
    score_tile_epilogue<KIND>(p, acc, q0, e0, tx, ty, cuts);
}

// ------------------------------------------------------------------------------------------
// score tile, kinds that are a function of (q, t) alone: the same 64 x 64 tile and the same
// operation order (one accumulator per pair, coordinates ascending), but the 64 query rows and
// 64 entity rows arrive by one asynchronous bulk copy per row into padded shared-memory rows (up
// to 128 coordinates per stage, two stages for longer rows), so a CTA waits once per stage instead
// of loading and synchronising every 32 coordinates.
// ------------------------------------------------------------------------------------------
constexpr int IKT = 128;
__host__ __device__ inline int infer_tma_kc(int d) { return d < IKT ? d : IKT; }
__host__ __device__ inline int infer_tma_stages(int d) { return d > IKT ? 2 : 1; }
inline size_t infer_tma_smem(int d) {
    return (size_t)infer_tma_stages(d) * (IQ + IE) * (infer_tma_kc(d) + 4) * sizeof(float) + 2 * sizeof(uint64_t);
}

// KC: the stage length when known at compile time (rows of at least IKT floats; shared-memory
// addresses of the inner loop are then constants off one base per operand), 0: shorter rows.
template <int KIND, int KC>
__global__ void __launch_bounds__(256) score_tile_tma_kernel(InferParams p) {
    extern __shared__ __align__(128) unsigned char smraw[];
    constexpr int ROWS = IQ + IE;        // rows [0, IQ) of a stage hold queries, the rest entities
    const int kc = KC ? KC : infer_tma_kc(p.d), ld = kc + 4, nstage = infer_tma_stages(p.d);
    const int nchunk = (p.d + kc - 1) / kc;
    float* base = reinterpret_cast<float*>(smraw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smraw + (size_t)nstage * ROWS * ld * sizeof(float));
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int qt = blockIdx.x % p.q_tiles;
    const int64_t et = blockIdx.x / p.q_tiles;
    const int q0 = qt * IQ;
    const int64_t e0 = p.e_lo + et * IE;

    if (tid == 0) {
        for (int st = 0; st < nstage; ++st) mbar_init(&bars[st], ROWS);
        mbar_init_fence();
    }
    __syncthreads();

    auto issue = [&](int chunk, int stage) {     // thread r < ROWS owns row r of the stage
        if (tid >= ROWS) return;
        const bool isq = tid < IQ;
        const int64_t g = isq ? q0 + tid : e0 + (tid - IQ);
        const bool in = isq ? g < p.nq : g < p.e_hi;
        float* dst = base + ((size_t)stage * ROWS + tid) * ld;
        const int k0 = chunk * kc, len = min(kc, p.d - k0);
        if (in) {
            const float* src = (isq ? p.w.iq : p.ent) + g * p.d + k0;
            mbar_arrive_expect_tx(&bars[stage], (uint32_t)len * 4u);
            bulk_g2s(dst, src, (uint32_t)len * 4u, &bars[stage]);
        } else {
            if (chunk < nstage)   // rows outside the problem stay zero for the whole kernel
                for (int k = 0; k < kc; k += 4) *reinterpret_cast<float4*>(dst + k) = make_float4(0.f, 0.f, 0.f, 0.f);
            mbar_arrive(&bars[stage]);
        }
    };
    issue(0, 0);
    if (nstage > 1 && nchunk > 1) issue(1, 1);
    __shared__ float4 cuts[IQ];
    if (tid >= 256 - IQ) score_tile_row_cuts(p, q0, e0, tid - (256 - IQ), cuts);     // (read after the barrier that follows the first wait)

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int chunk = 0; chunk < nchunk; ++chunk) {
        const int stage = chunk % nstage;
        const bool ok = mbar_wait_bounded(&bars[stage], (uint32_t)(chunk / nstage) & 1u, p.wait_limit);
        if (!__syncthreads_and(ok)) {
            if (tid == 0) set_status(p.w.status, KGE_ERR_TIMEOUT);
            // give copies still in flight a bounded chance to land before shared memory is released
            for (int st = 0; st < nstage; ++st) (void)mbar_wait_bounded(&bars[st], (uint32_t)(chunk / nstage) & 1u, p.wait_limit);
            return;
        }
        const float* Qs = base + (size_t)stage * ROWS * ld;
        const float* Ts = Qs + IQ * ld;
        const int len = min(kc, p.d - chunk * kc);
#pragma unroll 2
        for (int kk = 0; kk < len; kk += 4) {
            float4 qv[4], tv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                qv[i] = *reinterpret_cast<const float4*>(&Qs[(ty + 16 * i) * ld + kk]);
                tv[i] = *reinterpret_cast<const float4*>(&Ts[(tx + 16 * i) * ld + kk]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) canon_update<KIND>(acc[i][j], qv[i], tv[j]);
        }
        if (chunk + nstage < nchunk) {
            __syncthreads();             // every thread is done reading this stage
            issue(chunk + nstage, stage);
        }
    }
    score_tile_epilogue<KIND>(p, acc, q0, e0, tx, ty, cuts);
}

// ------------------------------------------------------------------------------------------
// The same score tile for rows of at least 128 floats, staged by the TMA engine's tensor copies:
// eight copies per stage (four 64-row x 32-float boxes of the queries, four of the entities, 128-byte
// swizzle) issued by one thread, instead of one bulk copy per row issued lane by lane (128 per
// tile, about 5 % of the kernel's instructions).  A box holds a row's 32 floats as eight 16-byte
// units, unit u of row r at position u ^ (r & 7): a thread's rows all share r & 7, so its eight
// unit offsets are computed once and every 128-bit read is base + constant + one of them, without
// bank conflicts.  What a box covers beyond the matrix reads as zero, and adding the term of a
// zero pair leaves every accumulator as it is, so ragged rows keep the canonical order and value.
// ------------------------------------------------------------------------------------------
constexpr int ITB_BOX_BYTES = 64 * 128, ITB_CHUNK_BYTES = 4 * ITB_BOX_BYTES, ITB_STAGE_BYTES = 2 * ITB_CHUNK_BYTES;
inline size_t infer_tensor_smem(int d) { return 1024 + (size_t)infer_tma_stages(d) * ITB_STAGE_BYTES + 2 * sizeof(uint64_t); }
__device__ __forceinline__ void tile_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

template <int KIND>
__global__ void __launch_bounds__(256, 3) score_tile_tensor_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmE,
                                                                   InferParams p) {
    extern __shared__ unsigned char smraw_t[];
    unsigned char* base = smraw_t + ((1024u - (smem_u32(smraw_t) & 1023u)) & 1023u);       // swizzled boxes want 1024-byte alignment
    const int nstage = infer_tma_stages(p.d);
    const int nchunk = (p.d + IKT - 1) / IKT;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)nstage * ITB_STAGE_BYTES);
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int qt = blockIdx.x % p.q_tiles;
    const int64_t et = blockIdx.x / p.q_tiles;
    const int q0 = qt * IQ;
    const int64_t e0 = p.e_lo + et * IE;

    if (tid == 0) {
        for (int st = 0; st < nstage; ++st) mbar_init(&bars[st], 1);
        mbar_init_fence();
    }
    __syncthreads();
    auto issue = [&](int chunk, int stage) {
        if (tid != 0) return;
        unsigned char* qs = base + (size_t)stage * ITB_STAGE_BYTES;
        mbar_arrive_expect_tx(&bars[stage], (uint32_t)ITB_STAGE_BYTES);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            tile_load_2d(qs + b * ITB_BOX_BYTES, &tmQ, chunk * IKT + 32 * b, q0, &bars[stage]);
            tile_load_2d(qs + ITB_CHUNK_BYTES + b * ITB_BOX_BYTES, &tmE, chunk * IKT + 32 * b, (int)e0, &bars[stage]);
        }
    };
    issue(0, 0);
    if (nstage > 1 && nchunk > 1) issue(1, 1);
    __shared__ float4 cuts[IQ];
    if (tid >= 256 - IQ) score_tile_row_cuts(p, q0, e0, tid - (256 - IQ), cuts);     // (read after the barrier that follows the first wait)

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    uint32_t qoff[8], toff[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { qoff[u] = (uint32_t)((u ^ (ty & 7)) << 4); toff[u] = (uint32_t)((u ^ (tx & 7)) << 4); }

    for (int chunk = 0; chunk < nchunk; ++chunk) {
        const int stage = chunk % nstage;
        const bool ok = mbar_wait_bounded(&bars[stage], (uint32_t)(chunk / nstage) & 1u, p.wait_limit);
        if (!__syncthreads_and(ok)) {
            if (tid == 0) set_status(p.w.status, KGE_ERR_TIMEOUT);
            for (int st = 0; st < nstage; ++st) (void)mbar_wait_bounded(&bars[st], (uint32_t)(chunk / nstage) & 1u, p.wait_limit);
            return;
        }
        const unsigned char* qrow = base + (size_t)stage * ITB_STAGE_BYTES + ty * 128;
        const unsigned char* trow = base + (size_t)stage * ITB_STAGE_BYTES + ITB_CHUNK_BYTES + tx * 128;
        const int nbox = (min(IKT, p.d - chunk * IKT) + 31) / 32;
#pragma unroll 1
        for (int b = 0; b < nbox; ++b) {
            const unsigned char* qb = qrow + b * ITB_BOX_BYTES;
            const unsigned char* tb = trow + b * ITB_BOX_BYTES;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float4 qv[4], tv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    qv[i] = *reinterpret_cast<const float4*>(qb + i * (16 * 128) + qoff[u]);
                    tv[i] = *reinterpret_cast<const float4*>(tb + i * (16 * 128) + toff[u]);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) canon_update<KIND>(acc[i][j], qv[i], tv[j]);
            }
        }
        if (chunk + nstage < nchunk) {
            __syncthreads();             // every thread is done reading this stage
            issue(chunk + nstage, stage);
        }
    }
    score_tile_epilogue<KIND>(p, acc, q0, e0, tx, ty, cuts);
}

template <int KIND>
cudaError_t launch_score_tile_tensor(const kge_handle* h, const InferParams& p, unsigned grid, cudaStream_t s) {
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        return cudaFuncSetAttribute(score_tile_tensor_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)infer_tensor_smem(kMaxDim));
    });
    if (e != cudaSuccess) return e;
    score_tile_tensor_kernel<KIND><<<grid, 256, infer_tensor_smem(p.d), s>>>(*reinterpret_cast<const CUtensorMap*>(h->tm_iq32),
                                                                            *reinterpret_cast<const CUtensorMap*>(h->tm_ent32), p);
    return cudaSuccess;
}

template <int KIND>
cudaError_t launch_score_tile_tma(const InferParams& p, unsigned grid, cudaStream_t s) {
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        const cudaError_t e0 = cudaFuncSetAttribute(score_tile_tma_kernel<KIND, IKT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)infer_tma_smem(kMaxDim));
        return e0 != cudaSuccess ? e0 : cudaFuncSetAttribute(score_tile_tma_kernel<KIND, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)infer_tma_smem(IKT));
    });
    if (e != cudaSuccess) return e;
    if (p.d >= IKT) score_tile_tma_kernel<KIND, IKT><<<grid, 256, infer_tma_smem(p.d), s>>>(p);
    else score_tile_tma_kernel<KIND, 0><<<grid, 256, infer_tma_smem(p.d), s>>>(p);
    return cudaSuccess;
}

// ------------------------------------------------------------------------------------------
// select: one CTA per query merges the running top-k with this chunk's candidates by a
// bitonic sort in shared memory under (score descending, id ascending), commits the chunk's
// rank count and resets the candidate list.
// ------------------------------------------------------------------------------------------
constexpr int SEL_THREADS = 128;
constexpr int SEL_MAX = 2 * kCandCap;   // k <= kCandCap plus at most kCandCap candidates

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(InferParams p) {
    __shared__ float ss[SEL_MAX];
    __shared__ int32_t si[SEL_MAX];
    const int q = blockIdx.x, tid = threadIdx.x;
    const int cnt = min(p.w.cand_cnt[q], kCandCap);
    const int total = p.k + cnt;
    int n2 = 1;
    while (n2 < total) n2 <<= 1;
    for (int i = tid; i < n2; i += SEL_THREADS) {
        float s = -INFINITY; int32_t id = INT_MAX;
        if (i < p.k) { s = p.w.top_score[(int64_t)q * p.k + i]; id = p.w.top_id[(int64_t)q * p.k + i]; }
        else if (i < total) { s = p.w.cand_score[(int64_t)q * kCandCap + i - p.k]; id = p.w.cand_id[(int64_t)q * kCandCap + i - p.k]; }
        ss[i] = s; si[i] = id;
    }
    __syncthreads();
    for (int size = 2; size <= n2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = tid; t < n2 / 2; t += SEL_THREADS) {
                const int lo = 2 * t - (t & (stride - 1)), hi = lo + stride;
                const bool up = (lo & size) == 0;   // "up" blocks end with the best element first
                const float a = ss[lo], b = ss[hi]; const int32_t ia = si[lo], ib = si[hi];
                const bool b_first = ordered_before(b, ib, a, ia);
                if (b_first == up) { ss[lo] = b; si[lo] = ib; ss[hi] = a; si[hi] = ia; }
            }
            __syncthreads();
        }
    }
    for (int i = tid; i < p.k; i += SEL_THREADS) {
        p.w.top_score[(int64_t)q * p.k + i] = ss[i];
        p.w.top_id[(int64_t)q * p.k + i] = si[i];
    }
    if (tid == 0) {
        p.w.thr[q] = ss[p.k - 1]; p.w.thr_id[q] = si[p.k - 1];
        p.w.beat[q] += p.w.beat_tmp[q];
        p.w.beat_tmp[q] = 0; p.w.cand_cnt[q] = 0;
    }
}

// Tensor-core inference: the true tail's score in the arithmetic of that path (operands rounded
// to bf16, fp32 accumulation), one thread per query.
__global__ void ftrue_bf16_kernel(InferParams p) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.nq || !p.tt) return;
    const uint16_t* qb = p.w.iqb + (int64_t)q * p.d;
    const uint16_t* tb = p.w.Eb + checked_id(p.tt[q], p.E, p.w.status) * p.d;
    float acc = 0.f;
    for (int k = 0; k < p.d; ++k)
        acc = __fmaf_rn(__uint_as_float((uint32_t)qb[k] << 16), __uint_as_float((uint32_t)tb[k] << 16), acc);
    p.w.iftrue[q] = acc;
}

// ---- sharded inference: the pieces that need rows of one shard only ----
// Query vectors of the queries whose head lies in this shard; zeros for the others, so that a sum over the shards
// (every head lies in exactly one) gives every query's vector exactly.
__global__ void shard_query_kernel(InferParams p, float* qvec_out, float* wh_scratch) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.nq) return;
    const int64_t hid = (int64_t)p.qh[q] - p.id_base;
    float* qv = qvec_out + (int64_t)q * p.d;
    if (hid < 0 || hid >= p.E) { for (int k = 0; k < p.d; ++k) qv[k] = 0.f; return; }
    const int64_t rid = checked_id(p.qr[q], p.R, p.w.status);
    build_query_seq(p, p.ent + hid * p.d, rid, qv, p.score == KGE_TRANSH ? wh_scratch + (int64_t)q * p.d : nullptr);
}

// Scores of the true tails that lie in this shard, from finished query vectors; zeros for the others.  bf16_rows: the
// tensor-core arithmetic (query vector and tail row rounded to bf16, fp32 accumulation).
__global__ void shard_ftrue_kernel(InferParams p, const float* qvec, float* wh_scratch, float* f_out, const uint16_t* bf16_rows) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.nq) return;
    const int64_t tid = (int64_t)p.tt[q] - p.id_base;
    if (tid < 0 || tid >= p.E) { f_out[q] = 0.f; return; }
    const float* qv = qvec + (int64_t)q * p.d;
    if (bf16_rows) {
        const uint16_t* tb = bf16_rows + tid * p.d;
        float acc = 0.f;
        for (int k = 0; k < p.d; ++k) {
            const __nv_bfloat16 qb = __float2bfloat16_rn(qv[k]);
            acc = __fmaf_rn(__bfloat162float(qb), __uint_as_float((uint32_t)tb[k] << 16), acc);
        }
        f_out[q] = acc;
        return;
    }
    float* wh = nullptr;
    if (p.score == KGE_TRANSH) { wh = wh_scratch + (int64_t)q * p.d; unit_normal_seq(p, checked_id(p.qr[q], p.R, p.w.status), wh); }
    f_out[q] = score_seq(p, qv, wh, p.ent + tid * p.d);
}

// Final top-k of a query over the candidates gathered from all shards: one CTA per query sorts per_query (score, id)
// pairs under (score descending, id ascending); unused places (id -1) sort last.
constexpr int MERGE_THREADS = 128, MERGE_MAX = 2048;
__global__ void __launch_bounds__(MERGE_THREADS) merge_topk_kernel(const int32_t* cand_ids, const float* cand_scores, int per_query, int k,
                                                                   int32_t* out_ids, float* out_scores) {
    __shared__ float ss[MERGE_MAX];
    __shared__ int32_t si[MERGE_MAX];
    const int q = blockIdx.x, tid = threadIdx.x;
    int n2 = 1;
    while (n2 < per_query) n2 <<= 1;
    for (int i = tid; i < n2; i += MERGE_THREADS) {
        float s = -INFINITY; int32_t id = INT_MAX;
        if (i < per_query) {
            id = cand_ids[(int64_t)q * per_query + i]; s = cand_scores[(int64_t)q * per_query + i];
            if (id < 0) { id = INT_MAX; s = -INFINITY; }
        }
        ss[i] = s; si[i] = id;
    }
    __syncthreads();
    for (int size = 2; size <= n2; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = tid; t < n2 / 2; t += MERGE_THREADS) {
                const int lo = 2 * t - (t & (stride - 1)), hi = lo + stride;
                const bool up = (lo & size) == 0;
                const float a = ss[lo], b = ss[hi]; const int32_t ia = si[lo], ib = si[hi];
                if (ordered_before(b, ib, a, ia) == up) { ss[lo] = b; si[lo] = ib; ss[hi] = a; si[hi] = ia; }
            }
            __syncthreads();
        }
    for (int i = tid; i < k; i += MERGE_THREADS) {
        const bool have = i < n2 && si[i] != INT_MAX;
        out_ids[(int64_t)q * k + i] = have ? si[i] : -1;
        out_scores[(int64_t)q * k + i] = have ? ss[i] : -INFINITY;
    }
}

__global__ void reset_chunk_kernel(InferParams p) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q < p.nq) { p.w.cand_cnt[q] = 0; p.w.beat_tmp[q] = 0; }
    if (q == 0) p.w.status[1] = 0;
}

__global__ void finish_kernel(InferParams p, int32_t* out_ids, float* out_scores, int32_t* out_ranks) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= p.nq) return;
    if (out_ids)
        for (int j = 0; j < p.k; ++j) {
            const int32_t id = p.w.top_id[(int64_t)q * p.k + j];
            out_ids[(int64_t)q * p.k + j] = id == INT_MAX ? -1 : id;
            out_scores[(int64_t)q * p.k + j] = p.w.top_score[(int64_t)q * p.k + j];
        }
    if (out_ranks) out_ranks[q] = (p.raw_beat ? 0 : 1) + p.w.beat[q];
}

cudaError_t launch_score_tiles(const kge_handle* h, const InferParams& p, cudaStream_t s) {
    const int64_t e_tiles = (p.e_hi - p.e_lo + IE - 1) / IE;
    const unsigned grid = (unsigned)(e_tiles * p.q_tiles);
    if (h->tiles32_ready && p.d >= IKT) {      // rows of at least 128 floats: tiles staged by tensor copies
        switch (p.kind) {
            case KIND_L1: return launch_score_tile_tensor<KIND_L1>(h, p, grid, s);
            case KIND_L2: return launch_score_tile_tensor<KIND_L2>(h, p, grid, s);
            case KIND_CL1: return launch_score_tile_tensor<KIND_CL1>(h, p, grid, s);
            case KIND_DOT: return launch_score_tile_tensor<KIND_DOT>(h, p, grid, s);
            default: break;
        }
    }
    switch (p.kind) {
        case KIND_L1: return launch_score_tile_tma<KIND_L1>(p, grid, s);
        case KIND_L2: return launch_score_tile_tma<KIND_L2>(p, grid, s);
        case KIND_CL1: return launch_score_tile_tma<KIND_CL1>(p, grid, s);
        case KIND_DOT: return launch_score_tile_tma<KIND_DOT>(p, grid, s);
        case KIND_TH_L1: score_tile_kernel<KIND_TH_L1><<<grid, 256, 0, s>>>(p); break;
        default: score_tile_kernel<KIND_TH_L2><<<grid, 256, 0, s>>>(p); break;
    }
    return cudaSuccess;
}

}  // namespace

namespace {
InferParams infer_params(kge_handle* h, const int32_t* qh, const int32_t* qr, int32_t nq, int32_t k, const int32_t* true_tails) {
    const kge_config& c = h->cfg;
    InferParams p;
    p.nq = nq; p.k = k; p.d = c.dim; p.d4 = c.dim / 4; p.score = c.score; p.kind = h->kind;
    p.E = c.num_entities; p.R = c.num_relations;
    p.ent = h->ent; p.rel = h->rel; p.relw = h->relw;
    p.qh = qh; p.qr = qr; p.tt = true_tails;
    p.q_tiles = (nq + IQ - 1) / IQ;
    p.wait_limit = h->wait_limit;
    p.id_base = 0; p.ext_q = nullptr; p.ext_ftrue = nullptr; p.raw_beat = 0;
    p.w = h->ws;
    p.e_lo = 0; p.e_hi = 0;
    return p;
}
}  // namespace

int run_shard_query_vectors(kge_handle* h, const int32_t* qh, const int32_t* qr, int32_t nq, int64_t ent_base, float* qvec_out, cudaStream_t s) {
    InferParams p = infer_params(h, qh, qr, nq, 1, nullptr);
    p.id_base = ent_base;
    shard_query_kernel<<<(nq + 127) / 128, 128, 0, s>>>(p, qvec_out, h->ws.iwhat);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

int run_shard_true_scores(kge_handle* h, const float* qvec, const int32_t* qr, const int32_t* true_tails, int32_t nq, int64_t ent_base,
                          float* ftrue_out, cudaStream_t s) {
    InferParams p = infer_params(h, nullptr, qr, nq, 1, true_tails);
    p.id_base = ent_base;
    if (h->ws.Eb && !h->eb_valid) {       // tensor-core arithmetic scores against the bf16 copy of the shard
        const int rc = launch_cast_bf16(h, h->ent, h->ws.Eb, h->cfg.num_entities * h->cfg.dim, s);
        if (rc != KGE_OK) return rc;
        h->eb_valid = true;
    }
    shard_ftrue_kernel<<<(nq + 127) / 128, 128, 0, s>>>(p, qvec, h->ws.iwhat, ftrue_out, h->ws.Eb);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

int run_merge_topk(const int32_t* cand_ids, const float* cand_scores, int32_t nq, int32_t per_query, int32_t k, int32_t* out_ids,
                   float* out_scores, cudaStream_t s) {
    if (per_query > MERGE_MAX) return KGE_ERR_WORKSPACE;
    merge_topk_kernel<<<nq, MERGE_THREADS, 0, s>>>(cand_ids, cand_scores, per_query, k, out_ids, out_scores);
    return cudaGetLastError() == cudaSuccess ? KGE_OK : KGE_ERR_CUDA;
}

int run_score_all_topk(kge_handle* h, const int32_t* qh, const int32_t* qr, int32_t nq, int32_t k,
                       const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                       cudaStream_t s, const ShardScoring* shard) {
    const kge_config& c = h->cfg;
    InferParams p = infer_params(h, qh, qr, nq, k, true_tails);
    if (shard) { p.id_base = shard->ent_base; p.ext_q = shard->qvec; p.ext_ftrue = shard->ftrue; p.raw_beat = 1; }
    const int qblocks = (nq + 127) / 128;
    query_setup_kernel<<<qblocks, 128, 0, s>>>(p);
    KGE_LAUNCH_CHECK(h);
    KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.status + 1, 0, 4, s));
    const bool tc = h->ws.Eb != nullptr;    // dot-product model with the tensor-core score block
    if (tc) {
        int rc = launch_cast_bf16(h, h->ws.iq, h->ws.iqb, (int64_t)nq * c.dim, s);
        if (rc == KGE_OK && !h->eb_valid) {     // the bf16 copy of the table is kept until the table changes
            rc = launch_cast_bf16(h, h->ent, h->ws.Eb, c.num_entities * c.dim, s);
            if (rc == KGE_OK) h->eb_valid = true;
        }
        if (rc != KGE_OK) return rc;
        if (!p.ext_ftrue) {
            ftrue_bf16_kernel<<<qblocks, 128, 0, s>>>(p);
            KGE_LAUNCH_CHECK(h);
        }
    }
    if (!tc && !h->tiles32_ready && c.dim >= IKT && h->kind != KIND_TH_L1 && h->kind != KIND_TH_L2) {
        // tensor maps of the fp32 query vectors and of the entity table (host-side encoding, nothing allocated)
        int rc = tc_make_f32_tile_map(h, h->tm_iq32, h->ws.iq, h->max_queries, c.dim);
        if (rc == KGE_OK) rc = tc_make_f32_tile_map(h, h->tm_ent32, h->ent, c.num_entities, c.dim);
        if (rc != KGE_OK) return rc;
        h->tiles32_ready = true;
    }
    auto score_chunk = [&](const InferParams& ip) -> int {
        if (tc) return launch_tc_infer_chunk(h, nq, ip.e_lo, ip.e_hi, true_tails, ip.id_base, s);
        KGE_CUDA_CHECK(h, launch_score_tiles(h, ip, s));
        KGE_LAUNCH_CHECK(h);
        return KGE_OK;
    };

    // Chunk i covers as many entities as all chunks before it (the first: one candidate
    // list's worth, since nothing is filtered yet), capped so a launch stays bounded.
    const int64_t max_chunk = std::max<int64_t>(kCandCap, std::min<int64_t>((int64_t)1 << 22, (int64_t)0x7fffffff / p.q_tiles * IE / 2));
    int64_t lo = 0;
    while (lo < p.E) {
        const int64_t len = std::min<int64_t>(std::min<int64_t>(std::max<int64_t>(lo, kCandCap), max_chunk), p.E - lo);
        p.e_lo = lo; p.e_hi = lo + len;
        { const int rc = score_chunk(p); if (rc != KGE_OK) return rc; }
        int32_t overflow = 0;
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(&overflow, h->ws.status + 1, 4, cudaMemcpyDeviceToHost, s));
        KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
        if (!overflow) {
            select_kernel<<<nq, SEL_THREADS, 0, s>>>(p);
            KGE_LAUNCH_CHECK(h);
        } else {
            // A list filled up (scores rising along the table): redo the chunk in pieces that
            // cannot overflow, selecting after each.
            reset_chunk_kernel<<<qblocks, 128, 0, s>>>(p);
            KGE_LAUNCH_CHECK(h);
            for (int64_t sub = lo; sub < lo + len; sub += kCandCap) {
                p.e_lo = sub; p.e_hi = std::min<int64_t>(sub + kCandCap, lo + len);
                { const int rc = score_chunk(p); if (rc != KGE_OK) return rc; }
                select_kernel<<<nq, SEL_THREADS, 0, s>>>(p);
                KGE_LAUNCH_CHECK(h);
            }
        }
        lo += len;
    }
    finish_kernel<<<qblocks, 128, 0, s>>>(p, out_ids, out_scores, out_ranks);
    KGE_LAUNCH_CHECK(h);
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return KGE_OK;
}

}  // namespace kge

// ------------------------------------------------------------------------------------------
// Full-entity scoring for callers that may not allocate device memory.  All scratch lives in
// one file-scope device array that every GPU loading the library holds until the process
// exits; nothing is allocated or freed here, on the host heap or on the device.
// ------------------------------------------------------------------------------------------
namespace kge {
namespace {

constexpr int kStaticMaxQueries = 64;
constexpr int kStaticMaxTopk = 32;
constexpr size_t kStaticQueryRows = (size_t)kStaticMaxQueries * kMaxDim * sizeof(float);       // 131072
constexpr size_t kStaticCandList = (size_t)kStaticMaxQueries * kCandCap * 4;                   // 262144
constexpr size_t kStaticTopList = (size_t)kStaticMaxQueries * kStaticMaxTopk * 4;              // 8192
constexpr size_t kStaticSmall = 256;                                                            // >= 64 x 4 bytes
constexpr size_t kStaticBytes = 256 + 2 * kStaticQueryRows + 6 * kStaticSmall + 2 * kStaticCandList + 2 * kStaticTopList;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];   // 804,608 bytes per GPU

constexpr int kStaticMaxDevices = 64;
void* g_static_scratch_addr[kStaticMaxDevices] = {};   // device address of the array, per device ordinal

}  // namespace
}  // namespace kge

extern "C" int kge_score_all_topk_static(const kge_config* cfg, const float* ent, const float* rel,
                                         const float* relw, const int32_t* q_heads, const int32_t* q_rels,
                                         int32_t nq, int32_t k, const int32_t* true_tails, int32_t* out_ids,
                                         float* out_scores, int32_t* out_ranks, void* stream) {
    using namespace kge;
    if (!cfg || !ent || !rel || !q_heads || !q_rels || !out_ids || !out_scores || nq < 0 || k <= 0)
        return KGE_ERR_BAD_ARG;
    if (out_ranks && !true_tails) return KGE_ERR_BAD_ARG;
    const kge_config& c = *cfg;
    if (c.num_entities <= 0 || c.num_entities > INT32_MAX || c.num_relations <= 0 || c.num_relations > INT32_MAX ||
        c.dim <= 0 || c.dim % 4 != 0 || c.score < KGE_TRANSE || c.score > KGE_ROTATE_REAL_L1 ||
        (c.p_norm != 1 && c.p_norm != 2) || (c.score == KGE_TRANSH && !relw))
        return KGE_ERR_BAD_ARG;
    // the fixed scratch bounds the problem: refuse anything it cannot hold
    if (nq > kStaticMaxQueries || k > kStaticMaxTopk || c.dim > kMaxDim) return KGE_ERR_WORKSPACE;
    if (nq == 0) return KGE_OK;

    kge_handle h{};                     // plain host object on the stack, every field zero; nothing in it is heap-backed
    h.cfg = c;
    h.kind = kind_of(c);
    if (c.score == KGE_ROTATE_REAL_L1) h.cfg.score = KGE_ROTATE;      // the same query vector, the real norm (see kge_create)
    h.kw = h.cfg.score == KGE_ROTATE ? c.dim / 2 : c.dim;
    h.ent = const_cast<float*>(ent); h.rel = const_cast<float*>(rel); h.relw = const_cast<float*>(relw);
    h.ent_state = h.rel_state = h.relw_state = nullptr;
    h.launches = 0; h.bound = true; h.graph_loaded = false;
    h.max_queries = kStaticMaxQueries; h.topk = kStaticMaxTopk;
    h.num_sms = 148; h.split_q = h.split_t = 1; h.num_triples = 0;
    h.ws_base = nullptr; h.ws_bytes = 0; h.streams_ready = false;
    h.wait_limit = kDefaultWaitLimit; h.capture_scores = nullptr;

    // Set-up, once per device and with that device current: in host code the array's name is
    // only a stand-in, so its device address has to be asked for.
    int dev = -1;
    KGE_CUDA_CHECK(&h, cudaGetDevice(&dev));
    if (dev < 0 || dev >= kStaticMaxDevices) return KGE_ERR_UNSUPPORTED;
    if (!g_static_scratch_addr[dev]) {
        void* addr = nullptr;
        KGE_CUDA_CHECK(&h, cudaGetSymbolAddress(&addr, g_static_scratch));
        g_static_scratch_addr[dev] = addr;
    }
    unsigned char* base = static_cast<unsigned char*>(g_static_scratch_addr[dev]);

    Workspace w{};
    size_t o = 0;
    auto take = [&](size_t bytes) { unsigned char* p = base + o; o += bytes; return p; };
    w.status = reinterpret_cast<int32_t*>(take(256));
    w.iq = reinterpret_cast<float*>(take(kStaticQueryRows));
    w.iwhat = reinterpret_cast<float*>(take(kStaticQueryRows));
    w.iftrue = reinterpret_cast<float*>(take(kStaticSmall));
    w.thr = reinterpret_cast<float*>(take(kStaticSmall));
    w.thr_id = reinterpret_cast<int32_t*>(take(kStaticSmall));
    w.cand_cnt = reinterpret_cast<int32_t*>(take(kStaticSmall));
    w.beat_tmp = reinterpret_cast<int32_t*>(take(kStaticSmall));
    w.beat = reinterpret_cast<int32_t*>(take(kStaticSmall));
    w.cand_score = reinterpret_cast<float*>(take(kStaticCandList));
    w.cand_id = reinterpret_cast<int32_t*>(take(kStaticCandList));
    w.top_score = reinterpret_cast<float*>(take(kStaticTopList));
    w.top_id = reinterpret_cast<int32_t*>(take(kStaticTopList));
    if (o != kStaticBytes) return KGE_ERR_WORKSPACE;
    h.ws = w;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array still holds the previous call's words: the status header must start at zero
    // (the per-query state is rewritten by the query set-up kernel)
    KGE_CUDA_CHECK(&h, cudaMemsetAsync(w.status, 0, 256, s));
    int rc = run_score_all_topk(&h, q_heads, q_rels, nq, k, true_tails, out_ids, out_scores, out_ranks, s, nullptr);
    if (rc != KGE_OK) return rc;
    int32_t word = 0;
    KGE_CUDA_CHECK(&h, cudaMemcpyAsync(&word, w.status, 4, cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(&h, cudaStreamSynchronize(s));
    return word;   // 0, or the code a kernel recorded (an id outside its table, a bounded wait that ran out)
}
