// Forward and backward of one shared-negative batch on CUDA cores (fp32):
//   build    : gather rows, per-query vectors q_b, positive scores, staged negative rows
//   block    : F[b,n] = f(q_b, t_n) for the whole B x N block (scoring-function table)
//   loss     : per-positive loss and dL/dF (Section 3.1 "Loss Functions"), in place
//   accum    : dQ_b = sum_n G_bn df/dq,  dT_n = sum_b G_bn df/dt  (owner computes, no atomics)
//   chain    : positive pair, chain rule q -> (h, r, w), reduction of the column splits
#include <cuda_bf16.h>

#include "kge_sample.cuh"

namespace kge {

namespace {

struct TrainParams {
    int B, N, d, d4, kw;
    int score, kind, loss;
    float gamma, adv_temp, ce_c, loss_scale;
    int64_t E, R;
    const float *ent, *rel, *relw;
    const int32_t *heads, *rels, *tails, *negs;
    int split_q, split_t;
    int th_slabs;          // TransH: slabs the tensor-core contractions append to dWpart and dTpart
    float* loss_out;    // caller's device scalar for the batch loss, or NULL
    int fused_sample;   // the gather kernel draws the batch itself (ids land in sp.heads ...) instead of reading it
    int slots_per_bucket;
    SampleParams sp;
    int tc_l2;          // TransE p = 2 with tensor-core backward: the splits hold C.T and C^T.Q, C = dL/dF / distance
    int neg_direct;     // the dT contraction wrote the negatives' gradient rows itself (one K split, no correction term)
    int wait_limit;     // tries of a bounded barrier wait
    const float* proj;  // feature-projection encoder: [2B+N, d] M e_F of the slots [heads | tails | negs], added to the rows read; or NULL
    float reg_lambda;   // L3 regulariser on the gathered entity rows (0 = off)
    int reg_form;       // 0: norms, 1: cubes
    Workspace w;
};

__device__ __forceinline__ float4 f4zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ float4 f4add(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }
__device__ __forceinline__ float4 f4sub(float4 a, float4 b) { return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w); }
__device__ __forceinline__ float4 f4mul(float4 a, float4 b) { return make_float4(a.x * b.x, a.y * b.y, a.z * b.z, a.w * b.w); }
__device__ __forceinline__ float4 f4scale(float s, float4 a) { return make_float4(s * a.x, s * a.y, s * a.z, s * a.w); }
__device__ __forceinline__ float4 f4fma(float s, float4 a, float4 c) {
    return make_float4(fmaf(s, a.x, c.x), fmaf(s, a.y, c.y), fmaf(s, a.z, c.z), fmaf(s, a.w, c.w));
}
__device__ __forceinline__ float f4dot(float4 a, float4 b) { return a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w; }
// L3 regulariser (Section 3.1 "Regularisation"): a lane's share of sum_k |e_k|^3, and c * e_k |e_k| (the gradient's shape).
__device__ __forceinline__ float f4cube(float4 a) {
    return fabsf(a.x) * a.x * a.x + fabsf(a.y) * a.y * a.y + fabsf(a.z) * a.z * a.z + fabsf(a.w) * a.w * a.w;
}
__device__ __forceinline__ float4 f4reg(float c, float4 a) {
    return make_float4(c * a.x * fabsf(a.x), c * a.y * fabsf(a.y), c * a.z * fabsf(a.z), c * a.w * fabsf(a.w));
}
// Factor of e_k |e_k| in the gradient of lambda * (term of one row) given s3 = sum_k |e_k|^3:
// norm: lambda / ||e||_3^2 (0 at e = 0); cube: 3 lambda.
__device__ __forceinline__ float reg_coef(float lambda, int form, float s3) {
    if (form == 1) return 3.f * lambda;
    if (!(s3 > 0.f)) return 0.f;
    const float n = cbrtf(s3);
    return lambda / (n * n);
}
// The sub-gradient of |x| that every p = 1 kernel of this library uses: +1 for x > 0, -1 otherwise.
// At x == 0 any value in [-1, 1] is a sub-gradient; the score-block backward counts the pairs with
// x > 0 (see add_if_gt), which fixes -1 there, and the positive pair takes the same value so that
// a step has one convention.
__device__ __forceinline__ float sgnf(float x) { return x > 0.f ? 1.f : -1.f; }
__device__ __forceinline__ float4 f4sgn(float4 a) { return make_float4(sgnf(a.x), sgnf(a.y), sgnf(a.z), sgnf(a.w)); }
// Four floats rounded to bf16 (nearest even), packed in memory order.
__device__ __forceinline__ uint2 pack_bf16x4(float4 v) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    return make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}


// ------------------------------------------------------------------------------------------
// build: one warp per row.  Warps [0, B) build q_b and f+_b; warps [B, B+N) stage t-_n.
// ------------------------------------------------------------------------------------------

// Per-lane contribution to the "distance accumulator" of a pair, for non-TransH kinds.
__device__ __forceinline__ float pair_partial(int kind, float4 q, float4 t) {
    if (kind == KIND_DOT) return f4dot(q, t);
    const float4 x = f4sub(q, t);
    if (kind == KIND_L1) return fabsf(x.x) + fabsf(x.y) + fabsf(x.z) + fabsf(x.w);
    if (kind == KIND_CL1) return sqrtf(fmaf(x.x, x.x, x.y * x.y)) + sqrtf(fmaf(x.z, x.z, x.w * x.w));
    return f4dot(x, x);
}

template <int kMaxChunks>   // float4 slices per lane: a warp owns a row
__global__ void __launch_bounds__(256) build_kernel(TrainParams p) {
    extern __shared__ uint64_t bucket_wcum[];   // fused sampling: cumulative weights of this CTA's bucket
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    allow_dependents();   // the score kernel may set up its shared memory while this one runs
    int64_t bucket_base = 0;
    if (p.fused_sample) {
        // The 8 query warps of a CTA draw from one triple bucket (the host checks that the slots
        // of a bucket are a multiple of 8): its cumulative weights are fetched side by side.
        const int w0 = blockIdx.x * (blockDim.x >> 5);
        if (w0 < p.B) {
            bucket_base = sample_bucket_base(p.sp, w0 / p.slots_per_bucket);
            if (p.sp.sample_mode == 0)
                for (int r = threadIdx.x; r <= (int)p.sp.R; r += blockDim.x) bucket_wcum[r] = p.sp.wcum[bucket_base + r];
        }
        __syncthreads();
    }
    if (warp >= p.B + p.N) return;
    const int d4 = p.d4;
    if (warp >= p.B) {
        const int n = warp - p.B;
        int32_t neg;
        if (p.fused_sample) { neg = sample_negative(p.sp, n); if (lane == 0) p.sp.negs[n] = neg; }
        else neg = p.negs[n];
        const int64_t id = checked_id(neg, p.E, p.w.status);
        const float4* src = reinterpret_cast<const float4*>(p.ent) + id * d4;
        float4* dst = reinterpret_cast<float4*>(p.w.Tneg) + (int64_t)n * d4;
        float nrm2 = 0.f, s3 = 0.f;
        const float4* pj = p.proj ? reinterpret_cast<const float4*>(p.proj) + (int64_t)(2 * p.B + n) * d4 : nullptr;
        for (int c = lane; c < d4; c += 32) {
            float4 v = src[c];
            if (pj) v = f4add(v, pj[c]);       // e = e_S + M_T e_F
            dst[c] = v;
            if (p.w.Tb) {   // tensor-core scoring: bf16 copy and the squared norm of the unrounded row
                reinterpret_cast<uint2*>(p.w.Tb)[(int64_t)n * d4 + c] = pack_bf16x4(v);
                nrm2 += f4dot(v, v);
            }
            if (p.w.reg_s3) s3 += f4cube(v);
        }
        if (p.w.Tb) { nrm2 = warp_sum(nrm2); if (lane == 0) p.w.tn2[n] = nrm2; }
        if (p.w.reg_s3) { s3 = warp_sum(s3); if (lane == 0) p.w.reg_s3[2 * p.B + n] = s3; }
        return;
    }
    const int b = warp;
    int32_t ih, ir, it;
    if (p.fused_sample) {
        if (lane == 0) {
            sample_positive(p.sp, b, bucket_base, bucket_wcum, ih, ir, it);
            p.sp.heads[b] = ih; p.sp.rels[b] = ir; p.sp.tails[b] = it;
        }
        ih = __shfl_sync(0xffffffffu, ih, 0); ir = __shfl_sync(0xffffffffu, ir, 0); it = __shfl_sync(0xffffffffu, it, 0);
    } else {
        ih = p.heads[b]; ir = p.rels[b]; it = p.tails[b];
    }
    const int64_t hid = checked_id(ih, p.E, p.w.status);
    const int64_t rid = checked_id(ir, p.R, p.w.status);
    const int64_t tid = checked_id(it, p.E, p.w.status);
    const float4* hrow = reinterpret_cast<const float4*>(p.ent) + hid * d4;
    const float4* trow = reinterpret_cast<const float4*>(p.ent) + tid * d4;
    float4 h[kMaxChunks], t[kMaxChunks], q[kMaxChunks], wh[kMaxChunks];
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) {
        const int c = lane + 32 * i;
        h[i] = c < d4 ? hrow[c] : f4zero();
        t[i] = c < d4 ? trow[c] : f4zero();
        if (p.proj && c < d4) {                // e = e_S + M_H e_F (head), e_S + M_T e_F (tail)
            h[i] = f4add(h[i], reinterpret_cast<const float4*>(p.proj)[(int64_t)b * d4 + c]);
            t[i] = f4add(t[i], reinterpret_cast<const float4*>(p.proj)[(int64_t)(p.B + b) * d4 + c]);
        }
        q[i] = f4zero(); wh[i] = f4zero();
    }
    if (p.w.reg_s3) {
        float sh = 0.f, st = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) { sh += f4cube(h[i]); st += f4cube(t[i]); }
        sh = warp_sum(sh); st = warp_sum(st);
        if (lane == 0) { p.w.reg_s3[b] = sh; p.w.reg_s3[p.B + b] = st; }
    }
    if (p.score == KGE_ROTATE) {
        const float2* th = reinterpret_cast<const float2*>(p.rel) + rid * d4;  // d/2 phases = d4 float2
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            if (c < d4) {
                const float2 ph = th[c];
                float s0, c0, s1, c1;
                sincosf(ph.x, &s0, &c0); sincosf(ph.y, &s1, &c1);
                q[i] = make_float4(h[i].x * c0 - h[i].y * s0, h[i].x * s0 + h[i].y * c0,
                                   h[i].z * c1 - h[i].w * s1, h[i].z * s1 + h[i].w * c1);
            }
        }
    } else {
        const float4* rrow = reinterpret_cast<const float4*>(p.rel) + rid * d4;
        float4 r[kMaxChunks];
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) { const int c = lane + 32 * i; r[i] = c < d4 ? rrow[c] : f4zero(); }
        if (p.score == KGE_TRANSE) {
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i) q[i] = f4add(h[i], r[i]);
        } else if (p.score == KGE_DISTMULT) {
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i) q[i] = f4mul(r[i], h[i]);
        } else if (p.score == KGE_COMPLEX) {
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i)
                q[i] = make_float4(r[i].x * h[i].x - r[i].y * h[i].y, r[i].x * h[i].y + r[i].y * h[i].x,
                                   r[i].z * h[i].z - r[i].w * h[i].w, r[i].z * h[i].w + r[i].w * h[i].z);
        } else {  // TransH: unit normal, projected head plus translation
            const float4* wrow = reinterpret_cast<const float4*>(p.relw) + rid * d4;
            float nrm2 = 0.f;
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i) {
                const int c = lane + 32 * i;
                wh[i] = c < d4 ? wrow[c] : f4zero();
                nrm2 += f4dot(wh[i], wh[i]);
            }
            const float inv = 1.f / fmaxf(sqrtf(warp_sum(nrm2)), 1e-12f);
            float a = 0.f;
            float ws = 0.f;
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i) {
                wh[i] = f4scale(inv, wh[i]); a += f4dot(wh[i], h[i]);
                ws += (wh[i].x + wh[i].y) + (wh[i].z + wh[i].w);
            }
            a = warp_sum(a); ws = warp_sum(ws);
            if (lane == 0) p.w.wsum[b] = ws;      // sum of the unit normal's coordinates (the p = 1 forward needs it per query)
#pragma unroll
            for (int i = 0; i < kMaxChunks; ++i) q[i] = f4add(f4fma(-a, wh[i], h[i]), r[i]);
        }
    }
    float4* qdst = reinterpret_cast<float4*>(p.w.Q) + (int64_t)b * d4;
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) { const int c = lane + 32 * i; if (c < d4) qdst[c] = q[i]; }
    if (p.w.Qb) {
        float nrm2 = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            if (c < d4) { reinterpret_cast<uint2*>(p.w.Qb)[(int64_t)b * d4 + c] = pack_bf16x4(q[i]); nrm2 += f4dot(q[i], q[i]); }
        }
        nrm2 = warp_sum(nrm2);
        if (lane == 0) p.w.qn2[b] = nrm2;
    }
    float acc = 0.f;
    if (p.score == KGE_TRANSH) {
        float4* wdst = reinterpret_cast<float4*>(p.w.What) + (int64_t)b * d4;
        float u = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            if (c < d4) wdst[c] = wh[i];
            u += f4dot(wh[i], t[i]);
        }
        u = warp_sum(u);
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const float4 x = f4fma(u, wh[i], f4sub(q[i], t[i]));
            acc += p.kind == KIND_TH_L1 ? fabsf(x.x) + fabsf(x.y) + fabsf(x.z) + fabsf(x.w) : f4dot(x, x);
        }
    } else {
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) acc += pair_partial(p.kind, q[i], t[i]);
    }
    acc = warp_sum(acc);
    if (lane == 0) {
        float f = acc;
        if (p.kind == KIND_L1 || p.kind == KIND_CL1 || p.kind == KIND_TH_L1) f = -acc;
        else if (p.kind == KIND_L2 || p.kind == KIND_TH_L2) f = -sqrtf(acc);
        p.w.fpos[b] = f;
    }
}

// ------------------------------------------------------------------------------------------
// block: F[b, n] = f(q_b, t_n).  Per-pair arithmetic of the kinds that are a function of
// (q, t) alone; the TransH block lives in kge_transh.cu.
// ------------------------------------------------------------------------------------------
constexpr int TN = 64;   // negative columns per score tile

__device__ __forceinline__ float approx_sqrt(float x) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float approx_rsqrt(float x) { float r; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

template <int KIND>
__device__ __forceinline__ void pair_update(float& acc, float4 q, float4 t) {
    if (KIND == KIND_DOT) {
        acc = fmaf(q.x, t.x, acc); acc = fmaf(q.y, t.y, acc); acc = fmaf(q.z, t.z, acc); acc = fmaf(q.w, t.w, acc);
    } else if (KIND == KIND_L1) {
        acc += fabsf(q.x - t.x); acc += fabsf(q.y - t.y); acc += fabsf(q.z - t.z); acc += fabsf(q.w - t.w);
    } else if (KIND == KIND_L2) {
        float x;
        x = q.x - t.x; acc = fmaf(x, x, acc); x = q.y - t.y; acc = fmaf(x, x, acc);
        x = q.z - t.z; acc = fmaf(x, x, acc); x = q.w - t.w; acc = fmaf(x, x, acc);
    } else {  // KIND_CL1: one special-function square root per complex component (relative error 2^-22)
        float xr = q.x - t.x, xi = q.y - t.y;
        acc += approx_sqrt(fmaf(xr, xr, xi * xi));
        xr = q.z - t.z; xi = q.w - t.w;
        acc += approx_sqrt(fmaf(xr, xr, xi * xi));
    }
}

// ------------------------------------------------------------------------------------------
// block, kinds that are a function of (q, t) alone: 32 x 64 pairs per CTA, 4 x 4 per thread.
// The 32 query rows and 64 negative rows of the tile are brought into shared memory by one
// asynchronous bulk copy per row (padded rows, so the 128-bit reads below are conflict-free),
// up to 128 floats of the embedding axis per stage, two stages when the rows are longer.
// ------------------------------------------------------------------------------------------
constexpr int FKC = 128;
constexpr int FTQ = 32;                  // query rows per tile
constexpr int FTHREADS = FTQ * 4;        // 4 x 4 pairs per thread, 64 negative columns per tile

__host__ __device__ inline int block_tma_kc(int d) { return d < FKC ? d : FKC; }
__host__ __device__ inline int block_tma_stages(int d) { return d > FKC ? 2 : 1; }
inline size_t block_tma_smem(int d) {
    return (size_t)block_tma_stages(d) * (FTQ + TN) * (block_tma_kc(d) + 4) * sizeof(float) + 2 * sizeof(uint64_t);
}

// KC: the stage length when it is known at compile time (rows of at least FKC floats): every
// shared-memory address of the inner loop is then one base per operand plus a constant, which
// removes two integer instructions per 128-bit load.  0: shorter rows, stage length = row length.
template <int KIND, int KC>
__global__ void __launch_bounds__(FTHREADS) block_tma_kernel(TrainParams p) {
    extern __shared__ __align__(128) unsigned char smraw[];
    constexpr int ROWS = FTQ + TN;       // rows [0, FTQ) of a stage hold queries, the rest negatives
    const int kc = KC ? KC : block_tma_kc(p.d), ld = kc + 4, nstage = block_tma_stages(p.d);
    const int nchunk = (p.d + kc - 1) / kc;
    float* base = reinterpret_cast<float*>(smraw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smraw + (size_t)nstage * ROWS * ld * sizeof(float));
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int b0 = blockIdx.y * FTQ, n0 = blockIdx.x * TN;

    if (tid == 0) {
        for (int st = 0; st < nstage; ++st) mbar_init(&bars[st], ROWS);
        mbar_init_fence();
    }
    __syncthreads();
    grid_dependency_wait();
    allow_dependents();

    auto issue = [&](int chunk, int stage) {     // thread r < ROWS owns row r of the stage
        if (tid >= ROWS) return;
        const bool isq = tid < FTQ;
        const int g = isq ? b0 + tid : n0 + tid - FTQ;
        float* dst = base + ((size_t)stage * ROWS + tid) * ld;
        const int k0 = chunk * kc, len = min(kc, p.d - k0);
        if (g < (isq ? p.B : p.N)) {
            const float* src = (isq ? p.w.Q : p.w.Tneg) + (int64_t)g * p.d + k0;
            mbar_arrive_expect_tx(&bars[stage], (uint32_t)len * 4u);
            bulk_g2s(dst, src, (uint32_t)len * 4u, &bars[stage]);
        } else {
            if (chunk < nstage)   // rows outside the problem stay zero for the whole kernel
                for (int k = 0; k < kc; k += 4) *reinterpret_cast<float4*>(dst + k) = f4zero();
            mbar_arrive(&bars[stage]);
        }
    };
    issue(0, 0);
    if (nstage > 1 && nchunk > 1) issue(1, 1);

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
        const float* Ts = Qs + FTQ * ld;
        const int len = min(kc, p.d - chunk * kc);
        // (measured: the plain L1 loop is fastest rolled, the others unrolled twice)
#pragma unroll (KIND == KIND_L1 ? 1 : 2)
        for (int kk = 0; kk < len; kk += 4) {
            float4 qv[4], tv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                qv[i] = *reinterpret_cast<const float4*>(&Qs[(ty + (FTQ / 4) * i) * ld + kk]);
                tv[i] = *reinterpret_cast<const float4*>(&Ts[(tx + 16 * i) * ld + kk]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) pair_update<KIND>(acc[i][j], qv[i], tv[j]);
        }
        if (chunk + nstage < nchunk) {
            __syncthreads();             // every thread is done reading this stage
            issue(chunk + nstage, stage);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int b = b0 + ty + (FTQ / 4) * i, n = n0 + tx + 16 * j;
            if (b >= p.B || n >= p.N) continue;
            float f = acc[i][j];
            if (KIND == KIND_L1 || KIND == KIND_CL1) f = -f;
            else if (KIND == KIND_L2) f = -sqrtf(f);
            p.w.F[(int64_t)b * p.N + n] = f;
        }
}

// ------------------------------------------------------------------------------------------
// loss: one CTA per positive.  The row of scores is read once into shared memory (rows too
// long for it are re-read from global memory), then overwritten with loss_scale * dL_b/dF_bn
// (divided by the distance for p = 2 kinds, which is the factor every later use needs).
// Also leaves the row sum of what it wrote, used by the TransE p = 1 backward.
// ------------------------------------------------------------------------------------------
constexpr int LOSS_THREADS = 256;
constexpr int LOSS_SMEM_FLOATS = 24 * 1024;   // rows up to 24,576 scores are staged in shared memory

__device__ __forceinline__ float block_sum(float v, float* sm) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sm[w] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < LOSS_THREADS / 32; ++i) t += sm[i];
    return t;
}
__device__ __forceinline__ float block_max(float v, float* sm) {
    v = warp_max(v);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sm[w] = v;
    __syncthreads();
    float t = sm[0];
    for (int i = 1; i < LOSS_THREADS / 32; ++i) t = fmaxf(t, sm[i]);
    return t;
}

// softplus(z) and sigmoid(z) from one exponential.  The special-function forms used here are good
// to a few 1e-7 absolute on softplus and a few 1e-6 relative on the exponentials, two orders below
// the tolerance of this path.
__device__ __forceinline__ void softplus_sigmoid(float z, float& sp, float& sg) {
    const float e = __expf(-fabsf(z));
    sp = fmaxf(z, 0.f) + __logf(1.f + e);
    const float r = __frcp_rn(1.f + e);
    sg = z >= 0.f ? r : e * r;
}

struct BlockReduce {   // all LOSS_THREADS threads of the CTA work on one row
    float* sm;
    __device__ __forceinline__ float sum(float v) const { return block_sum(v, sm); }
    __device__ __forceinline__ float max(float v) const { return block_max(v, sm); }
};
struct WarpReduce {    // one warp works on one row
    __device__ __forceinline__ float sum(float v) const { return warp_sum(v); }
    __device__ __forceinline__ float max(float v) const { return warp_max(v); }
};

template <int WPR>     // WPR neighbouring warps work on one row; every warp of the CTA calls each reduction
struct GroupReduce {
    float* sm;         // [2][warps of the CTA], the halves used in turn so that one barrier per reduction is enough
    int warp, lane;
    mutable int turn;
    template <class Op>
    __device__ __forceinline__ float across(float v, Op op) const {
        float* slot = sm + (turn & 1) * (LOSS_THREADS / 32);
        ++turn;
        if (lane == 0) slot[warp] = v;
        __syncthreads();
        const int first = warp / WPR * WPR;
        float t = slot[first];
#pragma unroll
        for (int i = 1; i < WPR; ++i) t = op(t, slot[first + i]);
        return t;
    }
    __device__ __forceinline__ float sum(float v) const { return across(warp_sum(v), [](float a, float c) { return a + c; }); }
    __device__ __forceinline__ float max(float v) const { return across(warp_max(v), [](float a, float c) { return fmaxf(a, c); }); }
};

// How a thread reaches its share of a row of scores: element i of count(), read with get(i),
// dL/dF written back with put(i, g).
struct StridedRow {    // scores in shared or global memory, covered as t0, t0 + stride, ...
    const float* row; float* out; int t0, stride, n;
    float* scratch;        // the staged copy of the row when it may be overwritten (shared memory), else NULL
    __device__ __forceinline__ int count() const { return n > t0 ? (n - t0 + stride - 1) / stride : 0; }
    __device__ __forceinline__ float get(int i) const { return row[t0 + i * stride]; }
    __device__ __forceinline__ void put(int i, float g) { out[t0 + i * stride] = g; }
    __device__ __forceinline__ bool can_keep() const { return scratch != nullptr; }
    __device__ __forceinline__ void keep(int i, float v) { scratch[t0 + i * stride] = v; }
    // the same row four scores at a time (a staged row of n % 4 == 0 scores, 16-byte aligned on both sides)
    __device__ __forceinline__ bool vec4() const { return scratch != nullptr && (n & 3) == 0; }
    __device__ __forceinline__ int count4() const { const int n4 = n >> 2; return n4 > t0 ? (n4 - t0 + stride - 1) / stride : 0; }
    __device__ __forceinline__ float4 get4(int i) const { return reinterpret_cast<const float4*>(row)[t0 + i * stride]; }
    __device__ __forceinline__ void keep4(int i, float4 v) { reinterpret_cast<float4*>(scratch)[t0 + i * stride] = v; }
    __device__ __forceinline__ void put4(int i, float4 g) { reinterpret_cast<float4*>(out)[t0 + i * stride] = g; }
};
template <int V4>      // scores in registers: V4 float4 per lane, the row is 128 * V4 long
struct RegisterRow {
    float4 f[V4], g[V4];
    __device__ __forceinline__ constexpr int count() const { return 4 * V4; }
    __device__ __forceinline__ float get(int i) const { return reinterpret_cast<const float*>(&f[i >> 2])[i & 3]; }
    __device__ __forceinline__ void put(int i, float v) { reinterpret_cast<float*>(&g[i >> 2])[i & 3] = v; }
    __device__ __forceinline__ constexpr bool can_keep() const { return false; }
    __device__ __forceinline__ void keep(int, float) {}
    __device__ __forceinline__ constexpr bool vec4() const { return false; }
    __device__ __forceinline__ constexpr int count4() const { return 0; }
    __device__ __forceinline__ float4 get4(int) const { return make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void keep4(int, float4) {}
    __device__ __forceinline__ void put4(int, float4) {}
};

// Loss and dL/dF of positive b over the calling threads' shares of the row; `lead` marks the
// one thread that writes the per-row scalars.
template <class Reduce, class Row>
__device__ __forceinline__ void loss_row(const TrainParams& p, int b, Row& row, bool lead, Reduce red) {
    const int N = p.N;
    const int cnt = row.count();
    const float fp = p.w.fpos[b];
    const bool l2 = p.kind == KIND_L2 || p.kind == KIND_TH_L2;
    const float ls = p.loss_scale;
    float gsum = 0.f;
    if (p.loss == KGE_LOSS_LOGSIGMOID) {
        const float a = p.adv_temp, gamma = p.gamma;
        float m = 0.f, z = (float)N;
        // Temperature exactly 1, a staged row and exp(gamma + m) finite: the weight's exponential e = exp(f - m) is kept in
        // the row's place, and exp(gamma + f) = K e with K = exp(gamma + m) gives the loss term and its derivative from it:
        // log(1 + K e) and K e / (1 + K e), three special-function instructions per score instead of five.
        bool shared_exp = false;
        if (a > 0.f) {
            const bool v4 = row.vec4();
            const int cnt4 = row.count4();
            float lm = -INFINITY;
            if (v4) {
                for (int i = 0; i < cnt4; ++i) { const float4 f = row.get4(i); lm = fmaxf(fmaxf(lm, a * f.x), fmaxf(fmaxf(a * f.y, a * f.z), a * f.w)); }
            } else {
#pragma unroll
                for (int i = 0; i < cnt; ++i) lm = fmaxf(lm, a * row.get(i));
            }
            m = red.max(lm);
            shared_exp = a == 1.f && !l2 && row.can_keep() && gamma + m <= 80.f;      // (the same for every thread of the row)
            float lz = 0.f;
            if (shared_exp && v4) {
                for (int i = 0; i < cnt4; ++i) {
                    const float4 f = row.get4(i);
                    const float4 e = make_float4(__expf(f.x - m), __expf(f.y - m), __expf(f.z - m), __expf(f.w - m));
                    row.keep4(i, e);
                    lz += (e.x + e.y) + (e.z + e.w);
                }
            } else if (shared_exp) {
                for (int i = 0; i < cnt; ++i) { const float e = __expf(row.get(i) - m); row.keep(i, e); lz += e; }
            } else {
#pragma unroll
                for (int i = 0; i < cnt; ++i) lz += __expf(a * row.get(i) - m);
            }
            z = red.sum(lz);
        }
        const float invz = 1.f / z;
        float lacc = 0.f;
        if (shared_exp && row.vec4()) {
            const float K = __expf(gamma + m);
            const int cnt4 = row.count4();
            for (int i = 0; i < cnt4; ++i) {
                const float4 e4 = row.get4(i);              // each thread reads back what it stored itself
                const float ev[4] = {e4.x, e4.y, e4.z, e4.w};
                float gv[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float t = K * ev[c], t1 = 1.f + t;
                    const float w = ev[c] * invz;
                    lacc += w * __logf(t1);
                    gv[c] = ls * w * __fdividef(t, t1);
                    gsum += gv[c];
                }
                row.put4(i, make_float4(gv[0], gv[1], gv[2], gv[3]));
            }
        } else if (shared_exp) {
            const float K = __expf(gamma + m);
            for (int i = 0; i < cnt; ++i) {
                const float e = row.get(i);                 // each thread reads back what it stored itself
                const float t = K * e, t1 = 1.f + t;
                const float w = e * invz;
                lacc += w * __logf(t1);
                const float g = ls * w * __fdividef(t, t1);       // (approximate reciprocal: 1 ulp, as in the tensor-core epilogues)
                row.put(i, g);
                gsum += g;
            }
        } else
#pragma unroll
        for (int i = 0; i < cnt; ++i) {
            const float f = row.get(i);
            const float w = a > 0.f ? __expf(a * f - m) * invz : invz;
            float sp, sg;
            softplus_sigmoid(gamma + f, sp, sg);
            lacc += w * sp;
            float g = ls * w * sg;
            if (l2) g = f < 0.f ? g / -f : 0.f;
            row.put(i, g);
            gsum += g;
        }
        const float lsum = red.sum(lacc);
        if (lead) {
            float sp, sg;
            softplus_sigmoid(-(gamma + fp), sp, sg);
            p.w.Lrow[b] = sp + lsum;
            p.w.gpos[b] = -ls * sg;
        }
    } else {
        const float c = p.ce_c;
        float lm = -INFINITY;
#pragma unroll
        for (int i = 0; i < cnt; ++i) lm = fmaxf(lm, row.get(i) + c);
        const float m = fmaxf(red.max(lm), fp);
        float lz = 0.f;
#pragma unroll
        for (int i = 0; i < cnt; ++i) lz += __expf(row.get(i) + c - m);
        const float epos = __expf(fp - m);
        const float z = red.sum(lz) + epos;
        const float invz = 1.f / z;
#pragma unroll
        for (int i = 0; i < cnt; ++i) {
            const float f = row.get(i);
            float g = ls * __expf(f + c - m) * invz;
            if (l2) g = f < 0.f ? g / -f : 0.f;
            row.put(i, g);
            gsum += g;
        }
        if (lead) {
            p.w.Lrow[b] = -fp + (m + logf(z));
            p.w.gpos[b] = ls * (epos * invz - 1.f);
        }
    }
    gsum = red.sum(gsum);
    if (lead) p.w.Grow[b] = gsum;
}

__device__ __forceinline__ void stage_row(float* dst, const float* src, int N, int t0, int stride) {
    if ((N & 3) == 0) {
        // eight loads in flight before the first store (load-then-store one at a time pays a trip to memory per element)
        const int n4 = N >> 2;
        for (int n = t0; n < n4; n += 8 * stride) {
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { const int idx = n + i * stride; v[i] = idx < n4 ? reinterpret_cast<const float4*>(src)[idx] : make_float4(0.f, 0.f, 0.f, 0.f); }
#pragma unroll
            for (int i = 0; i < 8; ++i) { const int idx = n + i * stride; if (idx < n4) reinterpret_cast<float4*>(dst)[idx] = v[i]; }
        }
    } else {
        for (int n = t0; n < N; n += stride) dst[n] = src[n];
    }
}

// One CTA per positive: long rows.
__global__ void __launch_bounds__(LOSS_THREADS) loss_kernel(TrainParams p) {
    extern __shared__ __align__(128) float rowbuf[];
    __shared__ float sm[LOSS_THREADS / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    grid_dependency_wait();
    allow_dependents();
    float* Frow = p.w.F + (int64_t)b * p.N;
    const float* row = Frow;
    if (p.N <= LOSS_SMEM_FLOATS) {
        if ((p.N & 3) == 0) {
            // the whole row as one bulk copy (a loop of load-then-store pays one trip to memory per 4 KB)
            __shared__ __align__(8) uint64_t bar;
            if (tid == 0) {
                mbar_init(&bar, 1);
                mbar_init_fence();
                mbar_arrive_expect_tx(&bar, (uint32_t)p.N * 4u);
                bulk_g2s(rowbuf, Frow, (uint32_t)p.N * 4u, &bar);
            }
            __syncthreads();                 // the barrier is initialised before anyone tests it
            const bool ok = mbar_wait_bounded(&bar, 0u, p.wait_limit);
            if (!__syncthreads_and(ok)) {
                if (tid == 0) { set_status(p.w.status, KGE_ERR_TIMEOUT); (void)mbar_wait_bounded(&bar, 0u, p.wait_limit); }
                return;
            }
        } else {
            stage_row(rowbuf, Frow, p.N, tid, LOSS_THREADS);
            __syncthreads();
        }
        row = rowbuf;
    }
    StridedRow sr{row, Frow, tid, LOSS_THREADS, p.N, p.N <= LOSS_SMEM_FLOATS ? rowbuf : nullptr};
    loss_row(p, b, sr, tid == 0, BlockReduce{sm});
}

// One warp per positive: rows of up to LOSS_WARP_MAX_N scores (N % 4 == 0), no CTA-wide barriers.
constexpr int LOSS_WARP_MAX_N = 2048;
__global__ void __launch_bounds__(LOSS_THREADS) loss_warp_kernel(TrainParams p) {
    extern __shared__ __align__(16) float rowbuf[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * (LOSS_THREADS / 32) + warp;
    grid_dependency_wait();
    allow_dependents();
    if (b >= p.B) return;
    float* Frow = p.w.F + (int64_t)b * p.N;
    float* row = rowbuf + (size_t)warp * p.N;
    stage_row(row, Frow, p.N, lane, 32);
    __syncwarp();
    StridedRow sr{row, Frow, lane, 32, p.N, row};
    loss_row(p, b, sr, lane == 0, WarpReduce{});
}

// WPR warps per positive with the whole row in registers (N = 128 * V4 * WPR): every pass over the
// row is unrolled, so the exponentials of a lane's 4 * V4 scores are independent instructions.
// With WPR > 1 the warps of a row exchange their partial maxima and sums through shared memory.
template <int V4, int WPR>
__global__ void __launch_bounds__(LOSS_THREADS) loss_reg_kernel(TrainParams p) {
    __shared__ float red_sm[2 * (LOSS_THREADS / 32)];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * (LOSS_THREADS / 32 / WPR) + warp / WPR, part = warp % WPR;
    grid_dependency_wait();
    allow_dependents();
    if (WPR == 1 && row >= p.B) return;
    const bool valid = row < p.B;
    const int b = valid ? row : p.B - 1;          // a CTA's spare warps shadow the last row: they take part in the barriers
    float4* Frow = reinterpret_cast<float4*>(p.w.F + (int64_t)b * p.N);
    RegisterRow<V4> rr;
#pragma unroll
    for (int j = 0; j < V4; ++j) rr.f[j] = Frow[(j * WPR + part) * 32 + lane];
    if (WPR == 1) loss_row(p, b, rr, lane == 0, WarpReduce{});
    else loss_row(p, b, rr, valid && part == 0 && lane == 0, GroupReduce<WPR>{red_sm, warp, lane, 0});
    if (valid) {
#pragma unroll
        for (int j = 0; j < V4; ++j) Frow[(j * WPR + part) * 32 + lane] = rr.g[j];
    }
}

// ------------------------------------------------------------------------------------------
// accum: out[r, :] = sum over the other side c of weight(r, c) * d f / d(owner row), for 32
// owner rows per CTA (4 per warp, a lane owns NCH float4 slices of the row) and one column
// split per blockIdx.y.  OWNER_Q: owner = queries (weights G[r, c]); else owner = negative
// tails (weights G[c, r]).  The sum runs over c ascending inside a split; the splits are
// added in ascending order by the chain kernel, so the result does not depend on timing.
// ------------------------------------------------------------------------------------------
struct AccArgs {
    const float *own, *oth;     // [own_rows, d], [oth_rows, d]
    const float *what;          // TransH: unit normals of the queries [B, d]
    const float *G, *U, *Cc;    // [B, N]
    int own_rows, oth_rows, N, d4, split;
    float *out, *out2;          // [split, own_rows, d]; out2: TransH normal gradient (OWNER_Q)
    float *csum;                // [split, own_rows] weight sums per owner row (TransE p = 1, owner = negatives)
    int32_t* status;
    int wait_limit;             // tries of a bounded barrier wait
};

constexpr int ACC_ROWS = 32, ACC_CC = 32, ACC_LDW = 36;

template <int KIND>
__device__ __forceinline__ void acc_update(float4& acc, float4 a, float4 b, float w) {
    if (KIND == KIND_DOT) {
        acc = f4fma(w, b, acc);
    } else if (KIND == KIND_L1) {  // acc -= w * sign(a - b), sign as in sgnf
        acc.x += a.x > b.x ? -w : w;
        acc.y += a.y > b.y ? -w : w;
        acc.z += a.z > b.z ? -w : w;
        acc.w += a.w > b.w ? -w : w;
    } else if (KIND == KIND_L2) {  // w already holds G / distance
        acc = f4fma(w, f4sub(b, a), acc);
    } else {                       // KIND_CL1: acc -= w * (a - b) / |a - b| per complex component
        // one special-function reciprocal square root per complex component (relative error 2^-22, as in the forward)
        float xr = a.x - b.x, xi = a.y - b.y, m2 = fmaf(xr, xr, xi * xi);
        // (a zero modulus has xr = xi = 0, so the finite factor from the floor contributes nothing)
        float s = w * approx_rsqrt(fmaxf(m2, 1e-37f));
        acc.x = fmaf(-s, xr, acc.x); acc.y = fmaf(-s, xi, acc.y);
        xr = a.z - b.z; xi = a.w - b.w; m2 = fmaf(xr, xr, xi * xi);
        s = w * approx_rsqrt(fmaxf(m2, 1e-37f));
        acc.z = fmaf(-s, xr, acc.z); acc.w = fmaf(-s, xi, acc.w);
    }
}

// ------------------------------------------------------------------------------------------
// accum, kinds that are a function of (q, t) alone.  Same ownership as above (32 owner rows
// per CTA, here 8 per warp, one column split per blockIdx.y), but the rows of the other side arrive
// 32 at a time by one asynchronous bulk copy into a double buffer, and the 32 x 32 weight tile
// of the next chunk is prefetched through registers while the current chunk is consumed.
//
// TransE p = 1: the term is w * sign(q - t).  Writing sign = 2 [q > t] - 1 (the value at an
// exact tie is a free choice of sub-gradient of |x| at 0; the whole step takes -1, see sgnf),
// the sum becomes 2 P - (sum of the weights) with
// P = sum of w over the pairs with q > t: one compare and one predicated add per element.
// The kernel accumulates P; the weight sums come from the loss kernel (rows) and from this
// kernel's own pass over the weight tiles (columns, OWNER_Q = false).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void add_if_gt(float& acc, float a, float b, float w) {
    asm("{\n .reg .pred p;\n setp.gt.f32 p, %1, %2;\n @p add.f32 %0, %0, %3;\n}\n" : "+f"(acc) : "f"(a), "f"(b), "f"(w));
}

template <int KIND, bool OWNER_Q>
__device__ __forceinline__ void acc_update2(float4& acc, float4 own, float4 oth, float w) {
    if (KIND == KIND_L1) {
        if (OWNER_Q) {   // own = q, oth = t
            add_if_gt(acc.x, own.x, oth.x, w); add_if_gt(acc.y, own.y, oth.y, w);
            add_if_gt(acc.z, own.z, oth.z, w); add_if_gt(acc.w, own.w, oth.w, w);
        } else {         // own = t, oth = q
            add_if_gt(acc.x, oth.x, own.x, w); add_if_gt(acc.y, oth.y, own.y, w);
            add_if_gt(acc.z, oth.z, own.z, w); add_if_gt(acc.w, oth.w, own.w, w);
        }
    } else {
        acc_update<KIND>(acc, own, oth, w);
    }
}

inline size_t accum_tma_smem(int d4) {
    return (size_t)2 * ACC_CC * d4 * 16 + (size_t)2 * ACC_CC * ACC_LDW * 4 + 8 * 32 * 4 + 2 * sizeof(uint64_t);
}

// ACC_WARPS warps per CTA, 32 / ACC_WARPS owner rows per warp (8 rows while the registers last).
// FULL: the rows are exactly 32 * NCH float4 long, so the row stride of the staged rows is a
// compile-time constant and no lane is idle.
template <int KIND, int NCH, bool OWNER_Q, int ACC_WARPS, bool FULL>
__device__ __forceinline__ void accum_tma_body(const AccArgs& a, const int block_x, const int block_y) {
    constexpr int ACC_RPW = ACC_ROWS / ACC_WARPS;
    constexpr int ACC_THREADS = 32 * ACC_WARPS;
    constexpr int ACC_WPT = ACC_ROWS * ACC_CC / ACC_THREADS;   // weights of a tile handled per thread
    extern __shared__ __align__(128) unsigned char smraw[];
    const int d4 = FULL ? 32 * NCH : a.d4;
    float4* Bs = reinterpret_cast<float4*>(smraw);                                  // [2][32][d4]
    float* Gs = reinterpret_cast<float*>(Bs + 2 * ACC_CC * d4);                     // [2][32][36], [c][r]
    float* Csum = Gs + 2 * ACC_CC * ACC_LDW;                                        // [warps][32]
    uint64_t* bars = reinterpret_cast<uint64_t*>(Csum + 8 * 32);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r0 = block_x * ACC_ROWS;
    const int per = ((a.oth_rows + a.split - 1) / a.split + ACC_CC - 1) / ACC_CC * ACC_CC;
    const int c_begin = block_y * per;
    const int c_end = min(a.oth_rows, c_begin + per);
    const int nchunk = c_end > c_begin ? (c_end - c_begin + ACC_CC - 1) / ACC_CC : 0;

    if (tid == 0) { mbar_init(&bars[0], 1); mbar_init(&bars[1], 1); mbar_init_fence(); }
    __syncthreads();
    grid_dependency_wait();
    allow_dependents();

    auto issue_rows = [&](int chunk, int buf) {      // thread 0 only
        const int c0 = c_begin + chunk * ACC_CC;
        const uint32_t bytes = (uint32_t)min(ACC_CC, c_end - c0) * (uint32_t)d4 * 16u;
        mbar_arrive_expect_tx(&bars[buf], bytes);
        bulk_g2s(Bs + (size_t)buf * ACC_CC * d4, reinterpret_cast<const float4*>(a.oth) + (int64_t)c0 * d4, bytes, &bars[buf]);
    };
    float greg[ACC_WPT];
    auto load_weights = [&](int chunk) {
        const int c0 = c_begin + chunk * ACC_CC;
#pragma unroll
        for (int e = 0; e < ACC_WPT; ++e) {
            const int idx = tid + ACC_THREADS * e;
            int rr, cc; int64_t g;
            if (OWNER_Q) { cc = idx & 31; rr = idx >> 5; g = (int64_t)(r0 + rr) * a.N + (c0 + cc); }
            else         { rr = idx & 31; cc = idx >> 5; g = (int64_t)(c0 + cc) * a.N + (r0 + rr); }
            greg[e] = ((r0 + rr) < a.own_rows && (c0 + cc) < c_end) ? a.G[g] : 0.f;
        }
    };
    auto store_weights = [&](int buf) {
#pragma unroll
        for (int e = 0; e < ACC_WPT; ++e) {
            const int idx = tid + ACC_THREADS * e;
            const int rr = OWNER_Q ? idx >> 5 : idx & 31, cc = OWNER_Q ? idx & 31 : idx >> 5;
            Gs[(buf * ACC_CC + cc) * ACC_LDW + rr] = greg[e];
        }
    };

    float4 A[ACC_RPW][NCH], acc[ACC_RPW][NCH];
#pragma unroll
    for (int i = 0; i < ACC_RPW; ++i)
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int r = r0 + warp * ACC_RPW + i, c = lane + 32 * j;
            A[i][j] = (r < a.own_rows && c < d4) ? reinterpret_cast<const float4*>(a.own)[(int64_t)r * d4 + c] : f4zero();
            acc[i][j] = f4zero();
        }
    float csum = 0.f;   // KIND_L1, owner = negatives: column (lane) sum of the weights this warp has seen

    if (nchunk > 0) {
        if (tid == 0) issue_rows(0, 0);
        load_weights(0);
        store_weights(0);
    }
    __syncthreads();
    for (int chunk = 0; chunk < nchunk; ++chunk) {
        const int cur = chunk & 1;
        const bool more = chunk + 1 < nchunk;
        if (more) {
            if (tid == 0) issue_rows(chunk + 1, cur ^ 1);
            load_weights(chunk + 1);
        }
        const bool ok = mbar_wait_bounded(&bars[cur], (uint32_t)(chunk >> 1) & 1u, a.wait_limit);
        if (!__syncthreads_and(ok)) {
            if (tid == 0) set_status(a.status, KGE_ERR_TIMEOUT);
            (void)mbar_wait_bounded(&bars[cur ^ 1], (uint32_t)((chunk + 1) >> 1) & 1u, a.wait_limit);
            return;
        }
        const int ccmax = min(ACC_CC, c_end - (c_begin + chunk * ACC_CC));
        const float4* Bc = Bs + (size_t)cur * ACC_CC * d4;
        const float* Gc = Gs + cur * ACC_CC * ACC_LDW;
        if (KIND == KIND_L1 && !OWNER_Q) {
#pragma unroll
            for (int e = 0; e < ACC_CC / ACC_WARPS; ++e) {
                const int cc = warp + ACC_WARPS * e;
                if (cc < ccmax) csum += Gc[cc * ACC_LDW + lane];
            }
        }
        // rolled: unrolled, the compiler holds the next iteration's operands in a second register set and copies them over
#pragma unroll 1
        for (int cc = 0; cc < ccmax; ++cc) {
            float gw[ACC_RPW];
#pragma unroll
            for (int i = 0; i < ACC_RPW; i += 4) {
                const float4 g4 = *reinterpret_cast<const float4*>(&Gc[cc * ACC_LDW + warp * ACC_RPW + i]);
                gw[i] = g4.x; gw[i + 1] = g4.y; gw[i + 2] = g4.z; gw[i + 3] = g4.w;
            }
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                const int c = lane + 32 * j;
                if (!FULL && c >= d4) continue;
                const float4 bv = Bc[cc * d4 + c];
#pragma unroll
                for (int i = 0; i < ACC_RPW; ++i) acc_update2<KIND, OWNER_Q>(acc[i][j], A[i][j], bv, gw[i]);
            }
        }
        if (more) store_weights(cur ^ 1);
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < ACC_RPW; ++i)
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int r = r0 + warp * ACC_RPW + i, c = lane + 32 * j;
            if (r >= a.own_rows || c >= d4) continue;
            reinterpret_cast<float4*>(a.out)[((int64_t)block_y * a.own_rows + r) * d4 + c] = acc[i][j];
        }
    if (KIND == KIND_L1 && !OWNER_Q) {
        Csum[warp * 32 + lane] = csum;
        __syncthreads();
        if (warp == 0 && r0 + lane < a.own_rows) {
            float t = 0.f;
            for (int w = 0; w < ACC_WARPS; ++w) t += Csum[w * 32 + lane];
            a.csum[(int64_t)block_y * a.own_rows + r0 + lane] = t;
        }
    }
}

// Both accumulations of a step in one launch: blockIdx.z = 0 owns query rows (dQ), 1 owns
// negative rows (dT); the grid spans the larger of the two shapes.
template <int KIND, int NCH, int ACC_WARPS, bool FULL>
__global__ void __launch_bounds__(32 * ACC_WARPS, NCH == 1 ? 4 : 1) accum_tma_kernel(AccArgs aq, AccArgs at) {
    const int own_rows = blockIdx.z == 0 ? aq.own_rows : at.own_rows, split = blockIdx.z == 0 ? aq.split : at.split;
    if ((int)blockIdx.x * ACC_ROWS >= own_rows || (int)blockIdx.y >= split) return;
    if (blockIdx.z == 0) accum_tma_body<KIND, NCH, true, ACC_WARPS, FULL>(aq, blockIdx.x, blockIdx.y);
    else accum_tma_body<KIND, NCH, false, ACC_WARPS, FULL>(at, blockIdx.x, blockIdx.y);
}

// ------------------------------------------------------------------------------------------
// chain: one warp per row (plus one CTA for the batch loss).  Warps [0, B): add the column splits of dQ (and of the TransH
// normal gradient), add the positive pair, apply the chain rule q -> (h, r, w) and write
// the gradient rows of the head, the positive tail and the relation.  Warps [B, B+N): add
// the row splits of dT and write the gradient row of the negative tail.
// ------------------------------------------------------------------------------------------
// Sum of n split partials first[0], first[stride], ... in ascending order.  Eight loads are issued
// before the first addition: a loop of load-then-add would pay one trip to L2 per split.
__device__ __forceinline__ float4 sum_splits(const float4* first, int64_t stride, int n) {
    float4 s = f4zero();
    for (int s0 = 0; s0 < n; s0 += 8) {
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = s0 + i < n ? first[(int64_t)(s0 + i) * stride] : f4zero();
#pragma unroll
        for (int i = 0; i < 8; ++i) s = f4add(s, v[i]);
    }
    return s;
}
__device__ __forceinline__ float sum_splits(const float* first, int64_t stride, int n) {
    float s = 0.f;
    for (int s0 = 0; s0 < n; s0 += 8) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = s0 + i < n ? first[(int64_t)(s0 + i) * stride] : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s += v[i];
    }
    return s;
}

template <int kMaxChunks>
__global__ void __launch_bounds__(256) chain_kernel(TrainParams p) {
    const int lane = threadIdx.x & 31;
    grid_dependency_wait();
    allow_dependents();
    if (blockIdx.x == gridDim.x - 1) {   // the extra last CTA adds up the batch loss
        __shared__ float lsum[8];
        float v = 0.f;
        for (int b = threadIdx.x; b < p.B; b += 256) v += p.w.Lrow[b];
        v *= p.loss_scale;
        if (p.w.reg_s3) {   // lambda Omega: one term per gathered row, added as it stands
            float om = 0.f;
            for (int i = threadIdx.x; i < 2 * p.B + p.N; i += 256) { const float s3 = p.w.reg_s3[i]; om += p.reg_form == 1 ? s3 : cbrtf(s3); }
            v = fmaf(p.reg_lambda, om, v);
        }
        v = warp_sum(v);
        if (lane == 0) lsum[threadIdx.x >> 5] = v;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int i = 0; i < 8; ++i) t += lsum[i];
            *p.w.loss = t;
            if (p.loss_out) *p.loss_out = t;
        }
        return;
    }
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= p.B + (p.neg_direct ? 0 : p.N)) return;
    const int d4 = p.d4;
    float4* gent = reinterpret_cast<float4*>(p.w.grad_ent);
    if (warp >= p.B) {
        const int n = warp - p.B;
        const float4* part = reinterpret_cast<const float4*>(p.w.dTpart);
        float wsum = 0.f;   // TransE p = 1: the splits hold P, the gradient is 2 P - (column sum of dL/dF)
        if (p.kind == KIND_L1) wsum = sum_splits(p.w.Cpart + n, p.N, p.split_t);
        const float creg = p.w.reg_s3 ? reg_coef(p.reg_lambda, p.reg_form, p.w.reg_s3[2 * p.B + n]) : 0.f;
        for (int c = lane; c < d4; c += 32) {
            float4 s = sum_splits(part + (int64_t)n * d4 + c, (int64_t)p.N * d4, p.split_t + p.th_slabs);
            if (p.kind == KIND_L1) s = make_float4(2.f * s.x - wsum, 2.f * s.y - wsum, 2.f * s.z - wsum, 2.f * s.w - wsum);
            if (p.tc_l2) {   // dT_n = sum_b C_bn (q_b - t_n) = (C^T Q)_n - (column sum of C) t_n
                const float cs = p.w.Gcol[n];
                const float4 t = reinterpret_cast<const float4*>(p.w.Tneg)[(int64_t)n * d4 + c];
                s = make_float4(s.x - cs * t.x, s.y - cs * t.y, s.z - cs * t.z, s.w - cs * t.w);
            }
            if (p.w.reg_s3) s = f4add(s, f4reg(creg, reinterpret_cast<const float4*>(p.w.Tneg)[(int64_t)n * d4 + c]));
            gent[(int64_t)(2 * p.B + n) * d4 + c] = s;
        }
        return;
    }
    const int b = warp;
    const int64_t hid = checked_id(p.heads[b], p.E, p.w.status);
    const int64_t rid = checked_id(p.rels[b], p.R, p.w.status);
    const int64_t tid = checked_id(p.tails[b], p.E, p.w.status);
    const float4* hrow = reinterpret_cast<const float4*>(p.ent) + hid * d4;
    const float4* trow = reinterpret_cast<const float4*>(p.ent) + tid * d4;
    const float4* qrow = reinterpret_cast<const float4*>(p.w.Q) + (int64_t)b * d4;
    const float gp = p.w.gpos[b], fp = p.w.fpos[b];

    float4 h[kMaxChunks], t[kMaxChunks], q[kMaxChunks], dq[kMaxChunks], dt[kMaxChunks];
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) {
        const int c = lane + 32 * i;
        const bool in = c < d4;
        h[i] = in ? hrow[c] : f4zero(); t[i] = in ? trow[c] : f4zero(); q[i] = in ? qrow[c] : f4zero();
        if (p.proj && in) {                    // the final embeddings, as the gather kernel formed them
            h[i] = f4add(h[i], reinterpret_cast<const float4*>(p.proj)[(int64_t)b * d4 + c]);
            t[i] = f4add(t[i], reinterpret_cast<const float4*>(p.proj)[(int64_t)(p.B + b) * d4 + c]);
        }
        float4 s = f4zero();
        if (in) s = sum_splits(reinterpret_cast<const float4*>(p.w.dQpart) + (int64_t)b * d4 + c, (int64_t)p.B * d4, p.split_q);
        if (p.kind == KIND_L1 && in) {   // the splits hold P; dQ = (row sum of dL/dF) - 2 P
            const float rs = p.w.Grow[b];
            s = make_float4(rs - 2.f * s.x, rs - 2.f * s.y, rs - 2.f * s.z, rs - 2.f * s.w);
        }
        if (p.tc_l2 && in) {             // dQ_b = sum_n C_bn (t_n - q_b) = (C T)_b - (row sum of C) q_b
            const float rs = p.w.Grow[b];
            s = make_float4(s.x - rs * q[i].x, s.y - rs * q[i].y, s.z - rs * q[i].z, s.w - rs * q[i].w);
        }
        dq[i] = s; dt[i] = f4zero();
    }
    float4* gh = gent + (int64_t)b * d4;
    float4* gt = gent + (int64_t)(p.B + b) * d4;
    // L3 regulariser: its gradient joins the head's and the positive tail's rows where they are stored
    const float creg_h = p.w.reg_s3 ? reg_coef(p.reg_lambda, p.reg_form, p.w.reg_s3[b]) : 0.f;
    const float creg_t = p.w.reg_s3 ? reg_coef(p.reg_lambda, p.reg_form, p.w.reg_s3[p.B + b]) : 0.f;

    if (p.score == KGE_TRANSH) {
        const float4* whrow = reinterpret_cast<const float4*>(p.w.What) + (int64_t)b * d4;
        const float4* wrow = reinterpret_cast<const float4*>(p.relw) + rid * d4;
        float4 wh[kMaxChunks], dwh[kMaxChunks];
        float u = 0.f, a = 0.f, nrm2 = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            const bool in = c < d4;
            wh[i] = in ? whrow[c] : f4zero();
            const float4 wraw = in ? wrow[c] : f4zero();
            nrm2 += f4dot(wraw, wraw);
            float4 s = f4zero();
            if (in) s = sum_splits(reinterpret_cast<const float4*>(p.w.dWpart) + (int64_t)b * d4 + c, (int64_t)p.B * d4, p.split_q + p.th_slabs);
            dwh[i] = s;
            u += f4dot(wh[i], t[i]); a += f4dot(wh[i], h[i]);
        }
        u = warp_sum(u); a = warp_sum(a); nrm2 = warp_sum(nrm2);
        // positive pair
        const float scale = p.kind == KIND_TH_L1 ? gp : (fp < 0.f ? gp / -fp : 0.f);
        float4 S[kMaxChunks];
        float cpos = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const float4 x = f4fma(u, wh[i], f4sub(q[i], t[i]));
            S[i] = p.kind == KIND_TH_L1 ? f4scale(-scale, f4sgn(x)) : f4scale(-scale, x);
            cpos += f4dot(S[i], wh[i]);
        }
        cpos = warp_sum(cpos);
        float wdq = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            dq[i] = f4add(dq[i], S[i]);
            dt[i] = f4fma(cpos, wh[i], f4scale(-1.f, S[i]));
            dwh[i] = f4fma(cpos, t[i], f4fma(u, S[i], dwh[i]));
            wdq += f4dot(wh[i], dq[i]);
        }
        wdq = warp_sum(wdq);
        // q = h - (w.h) w + r
        float wdw = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            dwh[i] = f4fma(-a, dq[i], f4fma(-wdq, h[i], dwh[i]));
            wdw += f4dot(wh[i], dwh[i]);
        }
        wdw = warp_sum(wdw);
        const float nrm = sqrtf(nrm2);
        const bool clamped = !(nrm > 1e-12f);
        const float inv = 1.f / fmaxf(nrm, 1e-12f);
        float4* gr = reinterpret_cast<float4*>(p.w.grad_rel) + (int64_t)b * d4;
        float4* gw = reinterpret_cast<float4*>(p.w.grad_relw) + (int64_t)b * d4;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            if (c >= d4) continue;
            gh[c] = f4add(f4fma(-wdq, wh[i], dq[i]), f4reg(creg_h, h[i]));
            gt[c] = f4add(dt[i], f4reg(creg_t, t[i]));
            gr[c] = dq[i];
            gw[c] = clamped ? f4scale(inv, dwh[i]) : f4scale(inv, f4fma(-wdw, wh[i], dwh[i]));
        }
        return;
    }

    // positive pair for the kinds whose pair is a function of (q, t) alone
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) {
        if (p.kind == KIND_DOT) {
            dq[i] = f4fma(gp, t[i], dq[i]);
            dt[i] = f4scale(gp, q[i]);
        } else if (p.kind == KIND_L1) {
            const float4 s = f4sgn(f4sub(q[i], t[i]));
            dq[i] = f4fma(-gp, s, dq[i]);
            dt[i] = f4scale(gp, s);
        } else if (p.kind == KIND_L2) {
            const float cpos = fp < 0.f ? gp / -fp : 0.f;
            const float4 x = f4sub(q[i], t[i]);
            dq[i] = f4fma(-cpos, x, dq[i]);
            dt[i] = f4scale(cpos, x);
        } else {  // KIND_CL1
            const float4 x = f4sub(q[i], t[i]);
            const float m0 = fmaf(x.x, x.x, x.y * x.y), m1 = fmaf(x.z, x.z, x.w * x.w);
            const float s0 = m0 > 0.f ? gp * rsqrtf(m0) : 0.f, s1 = m1 > 0.f ? gp * rsqrtf(m1) : 0.f;
            const float4 g = make_float4(s0 * x.x, s0 * x.y, s1 * x.z, s1 * x.w);
            dq[i] = f4sub(dq[i], g);
            dt[i] = g;
        }
    }
    if (p.score == KGE_ROTATE) {
        const float2* th = reinterpret_cast<const float2*>(p.rel) + rid * d4;
        float2* gr = reinterpret_cast<float2*>(p.w.grad_rel) + (int64_t)b * d4;
#pragma unroll
        for (int i = 0; i < kMaxChunks; ++i) {
            const int c = lane + 32 * i;
            if (c >= d4) continue;
            const float2 ph = th[c];
            float s0, c0, s1, c1;
            sincosf(ph.x, &s0, &c0); sincosf(ph.y, &s1, &c1);
            gh[c] = f4add(make_float4(dq[i].x * c0 + dq[i].y * s0, -dq[i].x * s0 + dq[i].y * c0,
                                      dq[i].z * c1 + dq[i].w * s1, -dq[i].z * s1 + dq[i].w * c1), f4reg(creg_h, h[i]));
            gt[c] = f4add(dt[i], f4reg(creg_t, t[i]));
            gr[c] = make_float2(-dq[i].x * q[i].y + dq[i].y * q[i].x, -dq[i].z * q[i].w + dq[i].w * q[i].z);
        }
        return;
    }
    const float4* rrow = reinterpret_cast<const float4*>(p.rel) + rid * d4;
    float4* gr = reinterpret_cast<float4*>(p.w.grad_rel) + (int64_t)b * d4;
#pragma unroll
    for (int i = 0; i < kMaxChunks; ++i) {
        const int c = lane + 32 * i;
        if (c >= d4) continue;
        gt[c] = f4add(dt[i], f4reg(creg_t, t[i]));
        const float4 rg = f4reg(creg_h, h[i]);
        if (p.score == KGE_TRANSE) {
            gh[c] = f4add(dq[i], rg); gr[c] = dq[i];
        } else if (p.score == KGE_DISTMULT) {
            const float4 r = rrow[c];
            gh[c] = f4add(f4mul(dq[i], r), rg); gr[c] = f4mul(dq[i], h[i]);
        } else {  // ComplEx: q = r * h
            const float4 r = rrow[c];
            gh[c] = f4add(make_float4(dq[i].x * r.x + dq[i].y * r.y, -dq[i].x * r.y + dq[i].y * r.x,
                                      dq[i].z * r.z + dq[i].w * r.w, -dq[i].z * r.w + dq[i].w * r.z), rg);
            gr[c] = make_float4(dq[i].x * h[i].x + dq[i].y * h[i].y, -dq[i].x * h[i].y + dq[i].y * h[i].x,
                                dq[i].z * h[i].z + dq[i].w * h[i].w, -dq[i].z * h[i].w + dq[i].w * h[i].z);
        }
    }
}

// ---- host-side dispatch ----
template <int KIND>
cudaError_t launch_block_tma(const TrainParams& p, cudaStream_t s) {
    const size_t smem = block_tma_smem(p.d);
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        const cudaError_t e0 = cudaFuncSetAttribute(block_tma_kernel<KIND, FKC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)block_tma_smem(kMaxDim));
        return e0 != cudaSuccess ? e0 : cudaFuncSetAttribute(block_tma_kernel<KIND, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)block_tma_smem(FKC));
    });
    if (e != cudaSuccess) return e;
    dim3 grid((p.N + TN - 1) / TN, (p.B + FTQ - 1) / FTQ);
    if (p.d >= FKC) return launch_dependent(block_tma_kernel<KIND, FKC>, grid, dim3(FTHREADS), smem, s, p);
    return launch_dependent(block_tma_kernel<KIND, 0>, grid, dim3(FTHREADS), smem, s, p);
}

template <int KIND, int NCH>
cudaError_t launch_accum_tma_inst(const AccArgs& aq, const AccArgs& at, cudaStream_t s) {
    constexpr int WARPS = NCH == 4 ? 8 : 4;
    const size_t smem = accum_tma_smem(aq.d4);
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        const cudaError_t e0 = cudaFuncSetAttribute(accum_tma_kernel<KIND, NCH, WARPS, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)accum_tma_smem(kMaxDim / 4));
        return e0 != cudaSuccess ? e0 : cudaFuncSetAttribute(accum_tma_kernel<KIND, NCH, WARPS, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                             (int)accum_tma_smem(kMaxDim / 4));
    });
    if (e != cudaSuccess) return e;
    dim3 grid((std::max(aq.own_rows, at.own_rows) + ACC_ROWS - 1) / ACC_ROWS, std::max(aq.split, at.split), 2);
    if (aq.d4 == 32 * NCH) return launch_dependent(accum_tma_kernel<KIND, NCH, WARPS, true>, grid, dim3(32 * WARPS), smem, s, aq, at);
    return launch_dependent(accum_tma_kernel<KIND, NCH, WARPS, false>, grid, dim3(32 * WARPS), smem, s, aq, at);
}

template <int KIND>
cudaError_t launch_accum_tma_kind(const AccArgs& aq, const AccArgs& at, cudaStream_t s) {
    if (aq.d4 <= 32) return launch_accum_tma_inst<KIND, 1>(aq, at, s);
    if (aq.d4 <= 64) return launch_accum_tma_inst<KIND, 2>(aq, at, s);
    return launch_accum_tma_inst<KIND, 4>(aq, at, s);
}

// dQ and dT of the pair kinds whose operands are plain rows, in one launch.
cudaError_t launch_accum_tma(int kind, const AccArgs& aq, const AccArgs& at, cudaStream_t s) {
    switch (kind) {
        case KIND_L1: return launch_accum_tma_kind<KIND_L1>(aq, at, s);
        case KIND_L2: return launch_accum_tma_kind<KIND_L2>(aq, at, s);
        case KIND_CL1: return launch_accum_tma_kind<KIND_CL1>(aq, at, s);
        default: return launch_accum_tma_kind<KIND_DOT>(aq, at, s);
    }
}

}  // namespace

int launch_forward_backward(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                            const int32_t* negs, float* loss_out, cudaStream_t s, cudaStream_t side, cudaStream_t dedup_side,
                            bool fused_sample, uint64_t step) {
    const kge_config& c = h->cfg;
    TrainParams p;
    p.B = c.batch; p.N = c.num_neg; p.d = c.dim; p.d4 = c.dim / 4; p.kw = h->kw;
    p.score = c.score; p.kind = h->kind; p.loss = c.loss;
    p.gamma = c.gamma; p.adv_temp = c.adv_temp; p.ce_c = c.ce_correction; p.loss_scale = c.loss_scale;
    p.E = c.num_entities; p.R = c.num_relations;
    p.ent = h->ent; p.rel = h->rel; p.relw = h->relw;
    p.heads = heads; p.rels = rels; p.tails = tails; p.negs = negs;
    p.split_q = h->split_q; p.split_t = h->split_t;
    p.th_slabs = th_contract_slabs(h);
    p.loss_out = loss_out;
    p.fused_sample = fused_sample ? 1 : 0;
    p.sp = make_sample_params(h, step);
    p.sp.heads = h->ws.heads; p.sp.rels = h->ws.rels; p.sp.tails = h->ws.tails; p.sp.negs = h->ws.negs;
    p.slots_per_bucket = c.batch / (c.head_part < 0 ? c.num_parts * c.num_parts : c.num_parts);
    p.tc_l2 = c.prec == KGE_PREC_BF16_TC && p.kind == KIND_L2;
    p.neg_direct = tc_negatives_direct(h) ? 1 : 0;
    p.wait_limit = h->wait_limit;
    p.reg_lambda = c.reg_lambda; p.reg_form = c.reg_form;
    p.proj = c.feat_dim > 0 ? h->ws.proj : nullptr;
    p.w = h->ws;
    const int nch = p.d4 <= 32 ? 1 : (p.d4 <= 64 ? 2 : 4);

    const int row_warps = p.B + p.N;
    stage_begin(h, ST_BUILD, s);
    {
        const int grid = (row_warps * 32 + 255) / 256;
        const size_t smem = fused_sample ? (size_t)(c.num_relations + 1) * 8 : 0;
        if (nch == 1) build_kernel<1><<<grid, 256, smem, s>>>(p);
        else if (nch == 2) build_kernel<2><<<grid, 256, smem, s>>>(p);
        else build_kernel<4><<<grid, 256, smem, s>>>(p);
    }
    stage_end(h, ST_BUILD, s);
    KGE_LAUNCH_CHECK(h);
    if (dedup_side) {
        // the batch ids are final: the sort of the touched ids runs beside everything up to the update
        KGE_CUDA_CHECK(h, cudaEventRecord(h->ev_ids, s));
        KGE_CUDA_CHECK(h, cudaStreamWaitEvent(dedup_side, h->ev_ids, 0));
        const int rc = launch_dedup(h, heads, rels, tails, negs, dedup_side);
        if (rc != KGE_OK) return rc;
        KGE_CUDA_CHECK(h, cudaEventRecord(h->ev_seg, dedup_side));
    }
    if (c.prec == KGE_PREC_BF16_TC) {
        // tensor cores: scores, loss and dL/dF in two fused passes, the score block never stored
        const int rc = launch_tc_forward(h, s);
        if (rc != KGE_OK) return rc;
    } else {
    stage_begin(h, ST_BLOCK, s);
    switch (p.kind) {
        case KIND_L1: KGE_CUDA_CHECK(h, launch_block_tma<KIND_L1>(p, s)); break;
        case KIND_L2: KGE_CUDA_CHECK(h, launch_block_tma<KIND_L2>(p, s)); break;
        case KIND_CL1: KGE_CUDA_CHECK(h, launch_block_tma<KIND_CL1>(p, s)); break;
        case KIND_DOT: KGE_CUDA_CHECK(h, launch_block_tma<KIND_DOT>(p, s)); break;
        default: { const int rc = launch_th_forward(h, s); if (rc != KGE_OK) return rc; h->launches -= 1; break; }   // TransH (counted below)
    }
    stage_end(h, ST_BLOCK, s);
    KGE_LAUNCH_CHECK(h);
    if (h->capture_scores)   // debug tap: the loss kernel is about to overwrite the scores in place
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(h->capture_scores, p.w.F, (size_t)p.B * p.N * sizeof(float), cudaMemcpyDeviceToDevice, s));
    stage_begin(h, ST_LOSS, s);
    {
        static DeviceOnce configured;
        KGE_CUDA_CHECK(h, once_per_device(configured, [] {
            const cudaError_t e = cudaFuncSetAttribute(loss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LOSS_SMEM_FLOATS * 4);
            if (e != cudaSuccess) return e;
            return cudaFuncSetAttribute(loss_warp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        LOSS_THREADS / 32 * LOSS_WARP_MAX_N * 4);
        }));
    }
    // rows of 256 / 512 / 1024 scores in registers, 2 / 4 / 4 warps per row (one warp per row leaves most of the SM idle:
    // 80 -> 75.5 us per step at B = N = 1024)
    constexpr int warps = LOSS_THREADS / 32;
    if (p.N == 256) KGE_CUDA_CHECK(h, (launch_dependent(loss_reg_kernel<1, 2>, dim3((p.B + warps / 2 - 1) / (warps / 2)), dim3(LOSS_THREADS), 0, s, p)));
    else if (p.N == 512) KGE_CUDA_CHECK(h, (launch_dependent(loss_reg_kernel<1, 4>, dim3((p.B + warps / 4 - 1) / (warps / 4)), dim3(LOSS_THREADS), 0, s, p)));
    else if (p.N == 1024) KGE_CUDA_CHECK(h, (launch_dependent(loss_reg_kernel<2, 4>, dim3((p.B + warps / 4 - 1) / (warps / 4)), dim3(LOSS_THREADS), 0, s, p)));
    else if (p.N <= LOSS_WARP_MAX_N && (p.N & 3) == 0) {
        constexpr int rows = LOSS_THREADS / 32;
        KGE_CUDA_CHECK(h, launch_dependent(loss_warp_kernel, dim3((p.B + rows - 1) / rows), dim3(LOSS_THREADS), (size_t)rows * p.N * 4, s, p));
    } else {
        KGE_CUDA_CHECK(h, launch_dependent(loss_kernel, dim3(p.B), dim3(LOSS_THREADS), p.N <= LOSS_SMEM_FLOATS ? (size_t)p.N * 4 : 0, s, p));
    }
    stage_end(h, ST_LOSS, s);
    KGE_LAUNCH_CHECK(h);
    }
    if (c.prec == KGE_PREC_BF16_TC) {
        const int rc = launch_tc_backward(h, s, side);
        if (rc != KGE_OK) return rc;
    } else {
    AccArgs aq;
    aq.own = p.w.Q; aq.oth = p.w.Tneg; aq.what = p.w.What; aq.G = p.w.F; aq.U = p.w.U; aq.Cc = p.w.Cc;
    aq.own_rows = p.B; aq.oth_rows = p.N; aq.N = p.N; aq.d4 = p.d4; aq.split = p.split_q;
    aq.out = p.w.dQpart; aq.out2 = p.w.dWpart; aq.csum = nullptr; aq.status = p.w.status; aq.wait_limit = h->wait_limit;
    AccArgs at = aq;
    at.own = p.w.Tneg; at.oth = p.w.Q; at.own_rows = p.N; at.oth_rows = p.B; at.split = p.split_t;
    at.out = p.w.dTpart; at.out2 = nullptr; at.csum = p.w.Cpart;
    if (p.kind != KIND_TH_L1 && p.kind != KIND_TH_L2) {
        // the two accumulations are independent: one launch holds both
        stage_begin(h, ST_ACCUM_Q, s);
        KGE_CUDA_CHECK(h, launch_accum_tma(p.kind, aq, at, s));
        stage_end(h, ST_ACCUM_Q, s);
        KGE_LAUNCH_CHECK(h);
    } else {
        // TransH: two launches, concurrent when there is a side stream
        if (side) {
            KGE_CUDA_CHECK(h, cudaEventRecord(h->ev_loss, s));
            KGE_CUDA_CHECK(h, cudaStreamWaitEvent(side, h->ev_loss, 0));
        }
        cudaStream_t sq = side ? side : s;
        { const int rc = launch_th_backward(h, sq, s); if (rc != KGE_OK) return rc; }
        if (side) {
            KGE_CUDA_CHECK(h, cudaEventRecord(h->ev_t, side));
            KGE_CUDA_CHECK(h, cudaStreamWaitEvent(s, h->ev_t, 0));
        }
    }
    }
    // the update follows the chain kernel directly: join the id sort here, where it has long finished
    if (dedup_side) KGE_CUDA_CHECK(h, cudaStreamWaitEvent(s, h->ev_seg, 0));
    stage_begin(h, ST_CHAIN, s);
    {
        const int grid = ((p.neg_direct ? p.B : row_warps) * 32 + 255) / 256 + 1;
        if (nch == 1) KGE_CUDA_CHECK(h, launch_dependent(chain_kernel<1>, dim3(grid), dim3(256), 0, s, p));
        else if (nch == 2) KGE_CUDA_CHECK(h, launch_dependent(chain_kernel<2>, dim3(grid), dim3(256), 0, s, p));
        else KGE_CUDA_CHECK(h, launch_dependent(chain_kernel<4>, dim3(grid), dim3(256), 0, s, p));
    }
    stage_end(h, ST_CHAIN, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
