// TransH score block and its backward on CUDA cores (scoring-function table, TransH row):
//   x_bnk = q_bk - t_nk + u_bn w_bk,   u_bn = w_b . t_n,   F_bn = -||x_bn||_p
// with w_b the unit normal of the query's relation and q_b the projected head plus translation.
// Every negative is projected per query, so the block is not a function of (q, t) alone:
//
//   forward   one kernel per 64 x 64 tile of pairs, two sweeps over the embedding axis with the
//             tile's rows resident in shared memory (bulk copies): first u, then the residual,
//             written as thr - t with thr = fma(u, w, q).  Besides F and u it leaves the pair's
//             contraction c'_bn = sum_k s_bnk w_bk (s = dF/dx up to sign: sign(x) for p = 1, x for
//             p = 2), which both backward kernels need as a finished number per pair: formed here
//             it costs two instructions per element, in a pass of its own it cost four.
//   backward  dq_b, dw_b (owner = query rows) and dt_n (owner = negative rows), one kernel each,
//             the other side's rows arriving 32 at a time by bulk copy into a double buffer and
//             the 32 x 32 tiles of per-pair numbers (dL/dF, u, c') prefetched through registers.
//             For p = 1 the sign is never formed: x > 0 is thr > t, one multiply-add and one
//             compare, and a sum of g sign(x) is 2 P - (sum of g) with P accumulated by
//             predicated adds (sign(0) = -1, the library's sub-gradient of |x| at 0).
//             Rows wider than 128 floats are cut into column slabs (blockIdx.z): given the
//             per-pair numbers every coordinate is independent of the others.
// Per element: 6 instructions forward (5 without the u sweep), 5 for the query side, 4 for the
// negatives' side.
//
// Three pieces of this are dense contractions and run on the tensor cores when the block is
// large enough (kge_handle::th_tc): u = W T^T forward, and in the backward the two sums whose
// coefficient is one number per pair, sum_n c_bn t_n and sum_b c_bn w_b with c = -dL/dF . c'.
// The operands are fp32, so each is split into bf16 terms (x = x1 + x2 + x3 for u, whose error
// moves the signs of the residuals; two terms for the backward sums) and the products that
// matter are accumulated in fp32: six for u (2^-25 relative per term), four for the others
// (2^-17).  The CUDA-core kernels then do 5, 4 and 3 instructions per element: the forward
// reads u instead of forming it, the query side writes c's split on its way.
#include "kge_common.cuh"
#include <cuda_bf16.h>

namespace kge {

namespace {

__device__ __forceinline__ float4 f4z() { return make_float4(0.f, 0.f, 0.f, 0.f); }
// acc += w where a > b: a compare into a predicate and a predicated add.  (A float mask, set.gt giving 1.0 or 0.0,
// times w in a multiply-add is the same count without the predicate registers and was measured 5-16 % slower.)
__device__ __forceinline__ void add_if_gt(float& acc, float a, float b, float w) {
    asm("{\n .reg .pred p;\n setp.gt.f32 p, %1, %2;\n @p add.f32 %0, %0, %3;\n}\n" : "+f"(acc) : "f"(a), "f"(b), "f"(w));
}
__device__ __forceinline__ void add2_if_gt(float& acc1, float& acc2, float a, float b, float w1, float w2) {
    asm("{\n .reg .pred p;\n setp.gt.f32 p, %2, %3;\n @p add.f32 %0, %0, %4;\n @p add.f32 %1, %1, %5;\n}\n"
        : "+f"(acc1), "+f"(acc2) : "f"(a), "f"(b), "f"(w1), "f"(w2));
}

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
constexpr int HB_Q = 64, HB_T = 64, HB_THREADS = 256, HB_KC = 128;      // (chunks of 64 floats were measured 4 % slower)
constexpr int HB_ROWS = 2 * HB_Q + HB_T;      // rows [0, 64) queries, [64, 128) their normals, [128, 192) negatives

struct ThFwdParams {
    int B, N, d;
    const float *Q, *What, *Tneg, *wsum;      // [B, d], [B, d], [N, d], [B] sum of the normal's coordinates
    float *F, *U, *Cp;                        // [B, N] score, w.t, c'
    int32_t* status;
    int wait_limit;
};

__host__ __device__ inline int hb_kc(int d) { return d < HB_KC ? d : HB_KC; }
__host__ __device__ inline int hb_stages(int d) { return d > HB_KC ? 2 : 1; }
inline size_t hb_smem(int d) { return (size_t)hb_stages(d) * HB_ROWS * (hb_kc(d) + 4) * sizeof(float) + 2 * sizeof(uint64_t); }

// KC: the chunk length when it is known at compile time (rows of at least HB_KC floats), so that
// every shared-memory address of the inner loops is one base per operand plus a constant; 0: rows
// shorter than HB_KC, chunk length = row length.
// UEXT: u = w.t is already in p.U (a tensor-core contraction wrote it): one sweep instead of two.
template <bool P1, int KC, bool UEXT>
__global__ void __launch_bounds__(HB_THREADS, 2) th_block_kernel(ThFwdParams p) {
    extern __shared__ __align__(128) unsigned char smraw[];
    const int kc = KC ? KC : hb_kc(p.d), ld = kc + 4, nstage = hb_stages(p.d);
    const int nchunk = (p.d + kc - 1) / kc;
    constexpr int SWEEP0 = UEXT ? 1 : 0;
    const bool resident = nchunk <= nstage;                     // every chunk has a stage of its own: loaded once, read by every sweep
    const int nload = resident ? nchunk : (2 - SWEEP0) * nchunk;   // else every sweep reads every chunk
    float* base = reinterpret_cast<float*>(smraw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smraw + (size_t)nstage * HB_ROWS * ld * sizeof(float));
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int b0 = blockIdx.y * HB_Q, n0 = blockIdx.x * HB_T;

    if (tid == 0) {
        for (int st = 0; st < nstage; ++st) mbar_init(&bars[st], HB_ROWS);
        mbar_init_fence();
    }
    __syncthreads();
    grid_dependency_wait();
    allow_dependents();

    auto issue = [&](int load, int stage) {      // thread r < HB_ROWS owns row r of the stage
        if (tid >= HB_ROWS) return;
        const int chunk = load % nchunk;
        const int kind = tid / HB_Q;             // 0 query, 1 normal, 2 negative
        const int g = kind == 2 ? n0 + tid - 2 * HB_Q : b0 + tid - kind * HB_Q;
        float* dst = base + ((size_t)stage * HB_ROWS + tid) * ld;
        const int k0 = chunk * kc, len = min(kc, p.d - k0);
        if (g < (kind == 2 ? p.N : p.B)) {
            const float* src = (kind == 0 ? p.Q : (kind == 1 ? p.What : p.Tneg)) + (int64_t)g * p.d + k0;
            mbar_arrive_expect_tx(&bars[stage], (uint32_t)len * 4u);
            bulk_g2s(dst, src, (uint32_t)len * 4u, &bars[stage]);
        } else {
            if (load < nstage)   // rows outside the problem stay zero for the whole kernel
                for (int k = 0; k < kc; k += 4) *reinterpret_cast<float4*>(dst + k) = f4z();
            mbar_arrive(&bars[stage]);
        }
    };
    issue(0, 0);
    if (nstage > 1) issue(1, 1);

    float acc[4][4], u[4][4], cw[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            acc[i][j] = 0.f; cw[i][j] = 0.f; u[i][j] = 0.f;
            if (UEXT) {
                const int b = b0 + ty + 16 * i, n = n0 + tx + 16 * j;
                if (b < p.B && n < p.N) u[i][j] = p.U[(int64_t)b * p.N + n];
            }
        }

    for (int sweep = SWEEP0; sweep < 2; ++sweep) {
        for (int chunk = 0; chunk < nchunk; ++chunk) {
            const int load = resident ? chunk : (sweep - SWEEP0) * nchunk + chunk;
            const int stage = load % nstage;
            const bool ok = mbar_wait_bounded(&bars[stage], (uint32_t)(load / nstage) & 1u, p.wait_limit);
            if (!__syncthreads_and(ok)) {
                if (tid == 0) set_status(p.status, KGE_ERR_TIMEOUT);
                // give copies still in flight a bounded chance to land before shared memory is released
                for (int st = 0; st < nstage; ++st) (void)mbar_wait_bounded(&bars[st], (uint32_t)(load / nstage) & 1u, p.wait_limit);
                return;
            }
            const float* Qs = base + (size_t)stage * HB_ROWS * ld;
            const float* Ws = Qs + HB_Q * ld;
            const float* Ts = Ws + HB_Q * ld;
            const int len = min(kc, p.d - chunk * kc);
            if (sweep == 0) {
#pragma unroll 2
                for (int kk = 0; kk < len; kk += 4) {
                    float4 wv[4], tv[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        wv[i] = *reinterpret_cast<const float4*>(&Ws[(ty + 16 * i) * ld + kk]);
                        tv[i] = *reinterpret_cast<const float4*>(&Ts[(tx + 16 * i) * ld + kk]);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            u[i][j] = fmaf(wv[i].x, tv[j].x, u[i][j]); u[i][j] = fmaf(wv[i].y, tv[j].y, u[i][j]);
                            u[i][j] = fmaf(wv[i].z, tv[j].z, u[i][j]); u[i][j] = fmaf(wv[i].w, tv[j].w, u[i][j]);
                        }
                }
            } else {
#pragma unroll 1
                for (int kk = 0; kk < len; kk += 4) {
                    float4 qv[4], wv[4], tv[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        qv[i] = *reinterpret_cast<const float4*>(&Qs[(ty + 16 * i) * ld + kk]);
                        wv[i] = *reinterpret_cast<const float4*>(&Ws[(ty + 16 * i) * ld + kk]);
                        tv[i] = *reinterpret_cast<const float4*>(&Ts[(tx + 16 * i) * ld + kk]);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float uu = u[i][j];
                            const float4 thr = make_float4(fmaf(uu, wv[i].x, qv[i].x), fmaf(uu, wv[i].y, qv[i].y),
                                                           fmaf(uu, wv[i].z, qv[i].z), fmaf(uu, wv[i].w, qv[i].w));
                            const float4 x = make_float4(thr.x - tv[j].x, thr.y - tv[j].y, thr.z - tv[j].z, thr.w - tv[j].w);
                            if (P1) {
                                acc[i][j] += fabsf(x.x); acc[i][j] += fabsf(x.y); acc[i][j] += fabsf(x.z); acc[i][j] += fabsf(x.w);
                                add_if_gt(cw[i][j], thr.x, tv[j].x, wv[i].x); add_if_gt(cw[i][j], thr.y, tv[j].y, wv[i].y);
                                add_if_gt(cw[i][j], thr.z, tv[j].z, wv[i].z); add_if_gt(cw[i][j], thr.w, tv[j].w, wv[i].w);
                            } else {
                                acc[i][j] = fmaf(x.x, x.x, acc[i][j]); acc[i][j] = fmaf(x.y, x.y, acc[i][j]);
                                acc[i][j] = fmaf(x.z, x.z, acc[i][j]); acc[i][j] = fmaf(x.w, x.w, acc[i][j]);
                                cw[i][j] = fmaf(x.x, wv[i].x, cw[i][j]); cw[i][j] = fmaf(x.y, wv[i].y, cw[i][j]);
                                cw[i][j] = fmaf(x.z, wv[i].z, cw[i][j]); cw[i][j] = fmaf(x.w, wv[i].w, cw[i][j]);
                            }
                        }
                }
            }
            if (!resident && load + nstage < nload) {
                __syncthreads();             // every thread is done reading this stage
                issue(load + nstage, stage);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int b = b0 + ty + 16 * i;
        if (b >= p.B) continue;
        const float ws = P1 ? p.wsum[b] : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx + 16 * j;
            if (n >= p.N) continue;
            const int64_t o = (int64_t)b * p.N + n;
            p.F[o] = P1 ? -acc[i][j] : -sqrtf(acc[i][j]);
            if (!UEXT) p.U[o] = u[i][j];
            p.Cp[o] = P1 ? 2.f * cw[i][j] - ws : cw[i][j];     // p = 1: cw holds the normal's coordinates summed where x > 0
        }
    }
}

// ------------------------------------------------------------------------------------------
// backward
// ------------------------------------------------------------------------------------------
constexpr int HA_CC = 32, HA_WARPS = 8, HA_THREADS = 32 * HA_WARPS;
// Owner rows per warp: four, or eight on the negatives' side once the c sums have left the kernel (one accumulator
// per row instead of two: the registers allow it, and an iteration's loads and loop instructions serve twice the arithmetic).
__host__ __device__ constexpr int ha_rpw(bool owner_q, bool tcc) { return (!owner_q && tcc) ? 8 : 4; }
constexpr int HA_SLAB = 128;                  // floats of a row handled by one thread block

struct ThAccArgs {
    const float *own, *oth;     // [own_rows, d], [oth_rows, d]
    const float *what;          // unit normals of the queries [B, d]
    const float *G, *U, *Cp;    // [B, N]: dL/dF (divided by the distance for p = 2), w.t, c'
    int own_rows, oth_rows, N, d, split;
    float *out, *out2;          // [split, own_rows, d]; out2: gradient of the unit normal (owner = queries)
    uint16_t* Csb;              // TCC, owner = queries: bf16 splits of c, [B, 2 ldc2] = [c1 | c2]
    int ldc2;                   // N rounded up to 64
    int32_t* status;
    int wait_limit;
};

// weight tiles of a chunk: g, u, then c (unless it goes to the tensor cores), then u g (query side)
__host__ __device__ constexpr int ha_tiles(bool owner_q, bool tcc) { return 2 + (tcc ? 0 : 1) + (owner_q ? 1 : 0); }
template <bool OWNER_Q, bool TCC>
inline size_t ha_smem() {
    constexpr int LDW = ha_rpw(OWNER_Q, TCC) * HA_WARPS + 4;
    return (size_t)2 * HA_CC * HA_SLAB * 4 * (OWNER_Q ? 1 : 2) + (size_t)2 * HA_CC * LDW * 4 * ha_tiles(OWNER_Q, TCC) + 2 * sizeof(uint64_t);
}

// OWNER_Q: owner rows are queries (own = Q, oth = Tneg); else negatives (own = Tneg, oth = Q, whose normals come along).
// The sums run over the other side's rows in ascending order inside a split; the chain kernel adds the splits in order.
// FULL_SLAB: every column slab is HA_SLAB floats wide (d a multiple of HA_SLAB), so the row stride
// of the staged rows is a compile-time constant.
// TCC: the sums with coefficient c are left to the tensor cores; the query side writes c's bf16 splits on its way.
template <bool P1, bool OWNER_Q, bool FULL_SLAB, bool TCC>
__global__ void __launch_bounds__(HA_THREADS, 2) th_accum_kernel(ThAccArgs a) {
    extern __shared__ __align__(128) unsigned char smraw[];
    constexpr int NT = ha_tiles(OWNER_Q, TCC);
    constexpr int HA_RPW = ha_rpw(OWNER_Q, TCC), HA_ROWS = HA_RPW * HA_WARPS, HA_LDW = HA_ROWS + 4;   // rows per warp / per block; tile row stride
    constexpr int HA_WPT = HA_ROWS * HA_CC / HA_THREADS, R4 = HA_RPW / 4;
    constexpr int TI_C = 2, TI_UG = TCC ? 2 : 3;             // tile indices behind g (0) and u (1)
    const int k0 = blockIdx.z * HA_SLAB, kc = FULL_SLAB ? HA_SLAB : min(HA_SLAB, a.d - k0), d4s = kc >> 2;
    float4* Bs = reinterpret_cast<float4*>(smraw);                                   // [2][32][d4s] rows of the other side
    float4* Ws = Bs + 2 * HA_CC * (HA_SLAB / 4);                                     // [2][32][d4s] their normals (owner = negatives)
    float* Tl = reinterpret_cast<float*>(Ws + (OWNER_Q ? 0 : 2 * HA_CC * (HA_SLAB / 4)));   // [2][NT][32][36] weight tiles, [c][r]
    uint64_t* bars = reinterpret_cast<uint64_t*>(Tl + 2 * NT * HA_CC * HA_LDW);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r0 = blockIdx.x * HA_ROWS;
    const int per = ((a.oth_rows + a.split - 1) / a.split + HA_CC - 1) / HA_CC * HA_CC;
    const int c_begin = blockIdx.y * per;
    const int c_end = min(a.oth_rows, c_begin + per);
    const int nchunk = c_end > c_begin ? (c_end - c_begin + HA_CC - 1) / HA_CC : 0;
    const bool whole = a.d == kc;                            // one slab: a chunk's rows are contiguous in memory

    if (tid == 0) { mbar_init(&bars[0], 1); mbar_init(&bars[1], 1); mbar_init_fence(); }
    __syncthreads();
    grid_dependency_wait();
    allow_dependents();

    auto issue_rows = [&](int chunk, int buf) {      // warp 0
        const int c0 = c_begin + chunk * HA_CC, cnt = min(HA_CC, c_end - c0);
        const uint32_t row_bytes = (uint32_t)kc * 4u;
        if (lane == 0) mbar_arrive_expect_tx(&bars[buf], (uint32_t)cnt * row_bytes * (OWNER_Q ? 1u : 2u));
        __syncwarp();
        float4* bdst = Bs + (size_t)buf * HA_CC * d4s;
        float4* wdst = Ws + (size_t)buf * HA_CC * d4s;
        if (whole) {
            if (lane == 0) {
                bulk_g2s(bdst, a.oth + (int64_t)c0 * a.d, (uint32_t)cnt * row_bytes, &bars[buf]);
                if (!OWNER_Q) bulk_g2s(wdst, a.what + (int64_t)c0 * a.d, (uint32_t)cnt * row_bytes, &bars[buf]);
            }
        } else if (lane < cnt) {
            bulk_g2s(bdst + (size_t)lane * d4s, a.oth + (int64_t)(c0 + lane) * a.d + k0, row_bytes, &bars[buf]);
            if (!OWNER_Q) bulk_g2s(wdst + (size_t)lane * d4s, a.what + (int64_t)(c0 + lane) * a.d + k0, row_bytes, &bars[buf]);
        }
    };
    float greg[HA_WPT], ureg[HA_WPT], creg[HA_WPT];
    auto load_weights = [&](int chunk) {
        const int c0 = c_begin + chunk * HA_CC;
#pragma unroll
        for (int e = 0; e < HA_WPT; ++e) {
            const int idx = tid + HA_THREADS * e;
            int rr, cc; int64_t g;
            if (OWNER_Q) { cc = idx & 31; rr = idx >> 5; g = (int64_t)(r0 + rr) * a.N + (c0 + cc); }
            else         { rr = idx & (HA_ROWS - 1); cc = idx / HA_ROWS; g = (int64_t)(c0 + cc) * a.N + (r0 + rr); }
            const bool in = (r0 + rr) < a.own_rows && (c0 + cc) < c_end;
            greg[e] = in ? a.G[g] : 0.f; ureg[e] = in ? a.U[g] : 0.f;
            if (!TCC || OWNER_Q) creg[e] = in ? a.Cp[g] : 0.f;
        }
    };
    auto store_weights = [&](int chunk, int buf) {
        float* T0 = Tl + (size_t)buf * NT * HA_CC * HA_LDW;
        const int c0 = c_begin + chunk * HA_CC;
#pragma unroll
        for (int e = 0; e < HA_WPT; ++e) {
            const int idx = tid + HA_THREADS * e;       // the element load_weights fetched
            const int rr = OWNER_Q ? idx >> 5 : idx & (HA_ROWS - 1), cc = OWNER_Q ? idx & 31 : idx / HA_ROWS;
            const int o = cc * HA_LDW + rr;
            T0[o] = greg[e];
            T0[HA_CC * HA_LDW + o] = ureg[e];
            if (!TCC) T0[TI_C * HA_CC * HA_LDW + o] = -greg[e] * creg[e];     // c_bn = -dL/dF . c'
            if (OWNER_Q) T0[TI_UG * HA_CC * HA_LDW + o] = ureg[e] * greg[e];
            if (TCC && OWNER_Q && blockIdx.z == 0 && (r0 + rr) < a.own_rows && (c0 + cc) < c_end) {
                // every pair passes here exactly once (in the first column slab): c = c1 + c2, two bf16 numbers
                const float c = -greg[e] * creg[e];
                const __nv_bfloat16 c1 = __float2bfloat16_rn(c), c2 = __float2bfloat16_rn(c - __bfloat162float(c1));
                uint16_t* dst = a.Csb + (int64_t)(r0 + rr) * (2 * a.ldc2) + (c0 + cc);
                dst[0] = __bfloat16_as_ushort(c1);
                dst[a.ldc2] = __bfloat16_as_ushort(c2);
            }
        }
    };

    const bool act = lane < d4s;
    // accumulators: acc; acc2 = the c sums (without TCC) or, for p = 2 on the query side, -sum u g x; acc3 = P weighted by u g (p = 1, query side)
    float4 A[HA_RPW], Wn[OWNER_Q ? HA_RPW : 1], acc[HA_RPW], acc2[HA_RPW], acc3[OWNER_Q ? HA_RPW : 1];
#pragma unroll
    for (int i = 0; i < HA_RPW; ++i) {
        const int r = r0 + warp * HA_RPW + i;
        const bool in = r < a.own_rows && act;
        A[i] = in ? *reinterpret_cast<const float4*>(a.own + (int64_t)r * a.d + k0 + 4 * lane) : f4z();
        if (OWNER_Q) { Wn[i] = in ? *reinterpret_cast<const float4*>(a.what + (int64_t)r * a.d + k0 + 4 * lane) : f4z(); acc3[i] = f4z(); }
        acc[i] = f4z(); acc2[i] = f4z();
    }
    float sg[HA_RPW], sug[HA_RPW];       // p = 1: this lane's share of the sums of g and of u g over the split, per owner row
#pragma unroll
    for (int i = 0; i < HA_RPW; ++i) { sg[i] = 0.f; sug[i] = 0.f; }

    if (nchunk > 0) {
        if (warp == 0) issue_rows(0, 0);
        load_weights(0);
        store_weights(0, 0);
    }
    __syncthreads();
    for (int chunk = 0; chunk < nchunk; ++chunk) {
        const int cur = chunk & 1;
        const bool more = chunk + 1 < nchunk;
        if (more) {
            if (warp == 0) issue_rows(chunk + 1, cur ^ 1);
            load_weights(chunk + 1);
        }
        const bool ok = mbar_wait_bounded(&bars[cur], (uint32_t)(chunk >> 1) & 1u, a.wait_limit);
        if (!__syncthreads_and(ok)) {
            if (tid == 0) set_status(a.status, KGE_ERR_TIMEOUT);
            (void)mbar_wait_bounded(&bars[cur ^ 1], (uint32_t)((chunk + 1) >> 1) & 1u, a.wait_limit);
            return;
        }
        const int ccmax = min(HA_CC, c_end - (c_begin + chunk * HA_CC));
        const float4* Bc = Bs + (size_t)cur * HA_CC * d4s;
        const float4* Wc = Ws + (size_t)cur * HA_CC * d4s;
        const float* Gc = Tl + (size_t)cur * NT * HA_CC * HA_LDW;
        const float* Uc = Gc + HA_CC * HA_LDW;
        const float* Cc = Gc + TI_C * HA_CC * HA_LDW;       // (not read with TCC)
        const float* UGc = Gc + TI_UG * HA_CC * HA_LDW;
        if (P1) {   // lane l adds the weights of the chunk's row l (rows beyond the chunk hold zeros)
#pragma unroll
            for (int h4 = 0; h4 < R4; ++h4) {
                const float4 g4 = *reinterpret_cast<const float4*>(&Gc[lane * HA_LDW + warp * HA_RPW + 4 * h4]);
                sg[4 * h4] += g4.x; sg[4 * h4 + 1] += g4.y; sg[4 * h4 + 2] += g4.z; sg[4 * h4 + 3] += g4.w;
                if (OWNER_Q) {
                    const float4 q4 = *reinterpret_cast<const float4*>(&UGc[lane * HA_LDW + warp * HA_RPW + 4 * h4]);
                    sug[4 * h4] += q4.x; sug[4 * h4 + 1] += q4.y; sug[4 * h4 + 2] += q4.z; sug[4 * h4 + 3] += q4.w;
                }
            }
        }
        if (act) {
            struct Operands { float4 g4[R4], u4[R4], c4[R4], q4[R4], bv, wv; };      // what one row of the other side brings
            auto fetch = [&](int cc) {
                Operands v;
#pragma unroll
                for (int h4 = 0; h4 < R4; ++h4) {
                    const int o = cc * HA_LDW + warp * HA_RPW + 4 * h4;
                    v.g4[h4] = *reinterpret_cast<const float4*>(&Gc[o]);
                    v.u4[h4] = *reinterpret_cast<const float4*>(&Uc[o]);
                    v.c4[h4] = TCC ? f4z() : *reinterpret_cast<const float4*>(&Cc[o]);
                    v.q4[h4] = OWNER_Q ? *reinterpret_cast<const float4*>(&UGc[o]) : f4z();
                }
                v.bv = Bc[cc * d4s + lane];
                v.wv = OWNER_Q ? f4z() : Wc[cc * d4s + lane];
                return v;
            };
            auto accumulate = [&](const Operands& v) {
                const float4 bv = v.bv;
                float gw[HA_RPW], uw[HA_RPW], cw[HA_RPW], ugw[HA_RPW];
#pragma unroll
                for (int h4 = 0; h4 < R4; ++h4) {
                    gw[4 * h4] = v.g4[h4].x; gw[4 * h4 + 1] = v.g4[h4].y; gw[4 * h4 + 2] = v.g4[h4].z; gw[4 * h4 + 3] = v.g4[h4].w;
                    uw[4 * h4] = v.u4[h4].x; uw[4 * h4 + 1] = v.u4[h4].y; uw[4 * h4 + 2] = v.u4[h4].z; uw[4 * h4 + 3] = v.u4[h4].w;
                    cw[4 * h4] = v.c4[h4].x; cw[4 * h4 + 1] = v.c4[h4].y; cw[4 * h4 + 2] = v.c4[h4].z; cw[4 * h4 + 3] = v.c4[h4].w;
                    ugw[4 * h4] = v.q4[h4].x; ugw[4 * h4 + 1] = v.q4[h4].y; ugw[4 * h4 + 2] = v.q4[h4].z; ugw[4 * h4 + 3] = v.q4[h4].w;
                }
                if (OWNER_Q) {       // own = q_b (A) with normal Wn; other = t_n (bv)
#pragma unroll
                    for (int i = 0; i < HA_RPW; ++i) {
                        const float4 thr = make_float4(fmaf(uw[i], Wn[i].x, A[i].x), fmaf(uw[i], Wn[i].y, A[i].y),
                                                       fmaf(uw[i], Wn[i].z, A[i].z), fmaf(uw[i], Wn[i].w, A[i].w));
                        if (P1) {    // acc = P (weights g), acc3 = P (weights u g), acc2 = sum of c t
                            add2_if_gt(acc[i].x, acc3[i].x, thr.x, bv.x, gw[i], ugw[i]); add2_if_gt(acc[i].y, acc3[i].y, thr.y, bv.y, gw[i], ugw[i]);
                            add2_if_gt(acc[i].z, acc3[i].z, thr.z, bv.z, gw[i], ugw[i]); add2_if_gt(acc[i].w, acc3[i].w, thr.w, bv.w, gw[i], ugw[i]);
                            if (!TCC) {
                                acc2[i].x = fmaf(cw[i], bv.x, acc2[i].x); acc2[i].y = fmaf(cw[i], bv.y, acc2[i].y);
                                acc2[i].z = fmaf(cw[i], bv.z, acc2[i].z); acc2[i].w = fmaf(cw[i], bv.w, acc2[i].w);
                            }
                        } else {     // acc = -sum g x, acc2 = sum (c t - u g x)
                            const float4 x = make_float4(thr.x - bv.x, thr.y - bv.y, thr.z - bv.z, thr.w - bv.w);
                            acc[i].x = fmaf(-gw[i], x.x, acc[i].x); acc[i].y = fmaf(-gw[i], x.y, acc[i].y);
                            acc[i].z = fmaf(-gw[i], x.z, acc[i].z); acc[i].w = fmaf(-gw[i], x.w, acc[i].w);
                            if (TCC) {
                                acc2[i].x = fmaf(-ugw[i], x.x, acc2[i].x); acc2[i].y = fmaf(-ugw[i], x.y, acc2[i].y);
                                acc2[i].z = fmaf(-ugw[i], x.z, acc2[i].z); acc2[i].w = fmaf(-ugw[i], x.w, acc2[i].w);
                            } else {
                                acc2[i].x = fmaf(cw[i], bv.x, fmaf(-ugw[i], x.x, acc2[i].x)); acc2[i].y = fmaf(cw[i], bv.y, fmaf(-ugw[i], x.y, acc2[i].y));
                                acc2[i].z = fmaf(cw[i], bv.z, fmaf(-ugw[i], x.z, acc2[i].z)); acc2[i].w = fmaf(cw[i], bv.w, fmaf(-ugw[i], x.w, acc2[i].w));
                            }
                        }
                    }
                } else {             // own = t_n (A); other = q_b (bv) with its normal wv
                    const float4 wv = v.wv;
#pragma unroll
                    for (int i = 0; i < HA_RPW; ++i) {
                        const float4 thr = make_float4(fmaf(uw[i], wv.x, bv.x), fmaf(uw[i], wv.y, bv.y), fmaf(uw[i], wv.z, bv.z), fmaf(uw[i], wv.w, bv.w));
                        if (P1) {    // acc = P (weights g), acc2 = sum of c w
                            add_if_gt(acc[i].x, thr.x, A[i].x, gw[i]); add_if_gt(acc[i].y, thr.y, A[i].y, gw[i]);
                            add_if_gt(acc[i].z, thr.z, A[i].z, gw[i]); add_if_gt(acc[i].w, thr.w, A[i].w, gw[i]);
                            if (!TCC) {
                                acc2[i].x = fmaf(cw[i], wv.x, acc2[i].x); acc2[i].y = fmaf(cw[i], wv.y, acc2[i].y);
                                acc2[i].z = fmaf(cw[i], wv.z, acc2[i].z); acc2[i].w = fmaf(cw[i], wv.w, acc2[i].w);
                            }
                        } else if (TCC) {   // acc = sum g x
                            acc[i].x = fmaf(gw[i], thr.x - A[i].x, acc[i].x); acc[i].y = fmaf(gw[i], thr.y - A[i].y, acc[i].y);
                            acc[i].z = fmaf(gw[i], thr.z - A[i].z, acc[i].z); acc[i].w = fmaf(gw[i], thr.w - A[i].w, acc[i].w);
                        } else {     // acc = sum (g x + c w)
                            acc[i].x = fmaf(cw[i], wv.x, fmaf(gw[i], thr.x - A[i].x, acc[i].x)); acc[i].y = fmaf(cw[i], wv.y, fmaf(gw[i], thr.y - A[i].y, acc[i].y));
                            acc[i].z = fmaf(cw[i], wv.z, fmaf(gw[i], thr.z - A[i].z, acc[i].z)); acc[i].w = fmaf(cw[i], wv.w, fmaf(gw[i], thr.w - A[i].w, acc[i].w));
                        }
                    }
                }
            };
            // Rolled, or unrolled completely; nothing in between.  With a loop left around two or more iterations the
            // compiler keeps the next iteration's loaded values in a second register set and copies them over (about 18
            // register moves per 80 arithmetic instructions, measured; unrolling by 2, 4, 8 or 16 was 1-10 % slower than
            // the rolled loop, two named operand sets taking turns 3-5 %).  Without any back edge there is nothing to
            // rotate: the query side with the c sums gone runs a full chunk's 32 iterations straight, 1.59 -> 1.48 ms at
            // B = N = 8192 (the negatives' side with eight rows per warp was 1 % slower that way and stays rolled).
            if (TCC && OWNER_Q && ccmax == HA_CC) {
#pragma unroll
                for (int cc = 0; cc < HA_CC; ++cc) accumulate(fetch(cc));
            } else {
#pragma unroll 1
                for (int cc = 0; cc < ccmax; ++cc) accumulate(fetch(cc));
            }
        }
        if (more) store_weights(chunk + 1, cur ^ 1);
        __syncthreads();
    }
    if (P1) {
#pragma unroll
        for (int i = 0; i < HA_RPW; ++i) { sg[i] = warp_sum(sg[i]); if (OWNER_Q) sug[i] = warp_sum(sug[i]); }
    }
#pragma unroll
    for (int i = 0; i < HA_RPW; ++i) {
        const int r = r0 + warp * HA_RPW + i;
        if (r >= a.own_rows || !act) continue;
        const int64_t o = ((int64_t)blockIdx.y * a.own_rows + r) * a.d + k0 + 4 * lane;
        float4 o1 = acc[i], o2 = acc2[i];
        if (P1) {
            const float4 P = acc[i], C = acc2[i];
            if (OWNER_Q) {   // -sum g sign(x) = (sum g) - 2 P;  sum (c t - u g sign(x)) = C - 2 P_u + (sum u g)
                const float4 Pu = acc3[OWNER_Q ? i : 0];
                o1 = make_float4(sg[i] - 2.f * P.x, sg[i] - 2.f * P.y, sg[i] - 2.f * P.z, sg[i] - 2.f * P.w);
                o2 = make_float4(C.x - 2.f * Pu.x + sug[i], C.y - 2.f * Pu.y + sug[i], C.z - 2.f * Pu.z + sug[i], C.w - 2.f * Pu.w + sug[i]);
            } else {         // sum (c w + g sign(x)) = C + 2 P - (sum g)
                o1 = make_float4(C.x + 2.f * P.x - sg[i], C.y + 2.f * P.y - sg[i], C.z + 2.f * P.z - sg[i], C.w + 2.f * P.w - sg[i]);
            }
        }
        *reinterpret_cast<float4*>(a.out + o) = o1;
        if (OWNER_Q) *reinterpret_cast<float4*>(a.out2 + o) = o2;
    }
}

template <bool P1, bool UEXT>
cudaError_t launch_fwd(const ThFwdParams& p, cudaStream_t s) {
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        const cudaError_t e0 = cudaFuncSetAttribute(th_block_kernel<P1, HB_KC, UEXT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hb_smem(kMaxDim));
        return e0 != cudaSuccess ? e0 : cudaFuncSetAttribute(th_block_kernel<P1, 0, UEXT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hb_smem(HB_KC));
    });
    if (e != cudaSuccess) return e;
    dim3 grid((p.N + HB_T - 1) / HB_T, (p.B + HB_Q - 1) / HB_Q);
    if (p.d >= HB_KC) return launch_dependent(th_block_kernel<P1, HB_KC, UEXT>, grid, dim3(HB_THREADS), hb_smem(p.d), s, p);
    return launch_dependent(th_block_kernel<P1, 0, UEXT>, grid, dim3(HB_THREADS), hb_smem(p.d), s, p);
}

// bf16 three-term splits x = x1 + x2 + x3 (2^-25 relative) of the unit normals and of the negatives, side by side:
// [rows, 3 dp] = [x1 | x2 | x3] with dp = d rounded up to 64 (the padding is zeroed once when the workspace is bound).
// One thread per four coordinates.
__global__ void __launch_bounds__(256) th_split3_kernel(const float4* W, int B, const float4* T, int N, int d4, int dp4, uint2* W3, uint2* T3) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)(B + N) * d4) return;
    const int row = (int)(i / d4), c = (int)(i - (int64_t)row * d4);
    const bool nrm = row < B;
    const float4 v = nrm ? W[i] : T[i - (int64_t)B * d4];
    const float x[4] = {v.x, v.y, v.z, v.w};
    uint16_t t1[4], t2[4], t3[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat16 a = __float2bfloat16_rn(x[e]);
        const float r1 = x[e] - __bfloat162float(a);
        const __nv_bfloat16 b = __float2bfloat16_rn(r1);
        const __nv_bfloat16 cc = __float2bfloat16_rn(r1 - __bfloat162float(b));
        t1[e] = __bfloat16_as_ushort(a); t2[e] = __bfloat16_as_ushort(b); t3[e] = __bfloat16_as_ushort(cc);
    }
    auto pack = [](const uint16_t* t) { return make_uint2((uint32_t)t[0] | ((uint32_t)t[1] << 16), (uint32_t)t[2] | ((uint32_t)t[3] << 16)); };
    uint2* dst = (nrm ? W3 + (int64_t)row * 3 * dp4 : T3 + (int64_t)(row - B) * 3 * dp4) + c;
    dst[0] = pack(t1); dst[dp4] = pack(t2); dst[2 * dp4] = pack(t3);
}

template <bool P1, bool OWNER_Q, bool TCC>
cudaError_t launch_acc(const ThAccArgs& a, cudaStream_t s) {
    static DeviceOnce configured;
    const cudaError_t e = once_per_device(configured, [] {
        const cudaError_t e0 = cudaFuncSetAttribute(th_accum_kernel<P1, OWNER_Q, true, TCC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ha_smem<OWNER_Q, TCC>());
        return e0 != cudaSuccess ? e0 : cudaFuncSetAttribute(th_accum_kernel<P1, OWNER_Q, false, TCC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ha_smem<OWNER_Q, TCC>());
    });
    if (e != cudaSuccess) return e;
    constexpr int rows = ha_rpw(OWNER_Q, TCC) * HA_WARPS;
    dim3 grid((a.own_rows + rows - 1) / rows, a.split, (a.d + HA_SLAB - 1) / HA_SLAB);
    if (a.d % HA_SLAB == 0) th_accum_kernel<P1, OWNER_Q, true, TCC><<<grid, HA_THREADS, ha_smem<OWNER_Q, TCC>(), s>>>(a);
    else th_accum_kernel<P1, OWNER_Q, false, TCC><<<grid, HA_THREADS, ha_smem<OWNER_Q, TCC>(), s>>>(a);
    return cudaSuccess;
}
template <bool OWNER_Q>
cudaError_t launch_acc_any(bool p1, bool tcc, const ThAccArgs& a, cudaStream_t s) {
    if (p1) return tcc ? launch_acc<true, OWNER_Q, true>(a, s) : launch_acc<true, OWNER_Q, false>(a, s);
    return tcc ? launch_acc<false, OWNER_Q, true>(a, s) : launch_acc<false, OWNER_Q, false>(a, s);
}

// bf16 two-term splits of the negatives and of the unit normals, [rows, 2d] = [x1 | x2]: the tensor-core
// contractions' second operands.  One thread per four coordinates.
__global__ void __launch_bounds__(256) th_split_rows_kernel(const float4* T, int N, const float4* W, int B, int d4, uint2* Ts, uint2* Ws) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)(N + B) * d4) return;
    const int row = (int)(i / d4), c = (int)(i - (int64_t)row * d4);
    const bool neg = row < N;
    const float4 v = neg ? T[i] : W[i - (int64_t)N * d4];
    uint2* dst = (neg ? Ts + (int64_t)row * 2 * d4 : Ws + (int64_t)(row - N) * 2 * d4) + c;
    const __nv_bfloat162 a1 = __floats2bfloat162_rn(v.x, v.y), b1 = __floats2bfloat162_rn(v.z, v.w);
    const float2 fa = __bfloat1622float2(a1), fb = __bfloat1622float2(b1);
    const __nv_bfloat162 a2 = __floats2bfloat162_rn(v.x - fa.x, v.y - fa.y), b2 = __floats2bfloat162_rn(v.z - fb.x, v.w - fb.y);
    dst[0] = make_uint2(*reinterpret_cast<const uint32_t*>(&a1), *reinterpret_cast<const uint32_t*>(&b1));
    dst[d4] = make_uint2(*reinterpret_cast<const uint32_t*>(&a2), *reinterpret_cast<const uint32_t*>(&b2));
}

}  // namespace

int launch_th_forward(kge_handle* h, cudaStream_t s) {
    const kge_config& c = h->cfg;
    const Workspace& w = h->ws;
    ThFwdParams p{c.batch, c.num_neg, c.dim, w.Q, w.What, w.Tneg, w.wsum, w.F, w.U, w.Cc, w.status, h->wait_limit};
    const bool p1 = h->kind == KIND_TH_L1;
    if (h->th_tc) {
        // u = w.t for all pairs as one tensor-core contraction over the operands' three-term splits (six products per K slice)
        stage_begin(h, ST_TH_U, s);
        const int64_t n4 = (int64_t)(c.batch + c.num_neg) * (c.dim / 4);
        const int dp = (c.dim + 63) / 64 * 64;
        th_split3_kernel<<<(int)((n4 + 255) / 256), 256, 0, s>>>(reinterpret_cast<const float4*>(w.What), c.batch,
                                                                 reinterpret_cast<const float4*>(w.Tneg), c.num_neg, c.dim / 4, dp / 4,
                                                                 reinterpret_cast<uint2*>(w.W3b), reinterpret_cast<uint2*>(w.T3b));
        KGE_LAUNCH_CHECK(h);
        const int rc = launch_tc_gemm_terms(h, h->tm_w3, h->tm_t3, c.batch, c.num_neg, dp, w.U, c.num_neg, s);
        if (rc != KGE_OK) return rc;
        stage_end(h, ST_TH_U, s);
        stage_begin(h, ST_BLOCK, s);      // (the caller's bracket opened before the contraction: open it again here)
        KGE_CUDA_CHECK(h, p1 ? (launch_fwd<true, true>(p, s)) : (launch_fwd<false, true>(p, s)));
    } else {
        KGE_CUDA_CHECK(h, p1 ? (launch_fwd<true, false>(p, s)) : (launch_fwd<false, false>(p, s)));
    }
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

// dQ / dW on `sq`, dT on `st` (the same stream, or two streams the caller has ordered after the loss kernel).
int launch_th_backward(kge_handle* h, cudaStream_t sq, cudaStream_t st) {
    const kge_config& c = h->cfg;
    const Workspace& w = h->ws;
    const bool p1 = h->kind == KIND_TH_L1;
    ThAccArgs aq{w.Q, w.Tneg, w.What, w.F, w.U, w.Cc, c.batch, c.num_neg, c.num_neg, c.dim, h->split_q, w.dQpart, w.dWpart,
                 w.Csb, (c.num_neg + 63) / 64 * 64, w.status, h->wait_limit};
    ThAccArgs at = aq;
    at.own = w.Tneg; at.oth = w.Q; at.own_rows = c.num_neg; at.oth_rows = c.batch; at.split = h->split_t;
    at.out = w.dTpart; at.out2 = nullptr;
    const bool tcc = h->th_tc;
    stage_begin(h, ST_ACCUM_Q, sq);
    if (tcc) {      // second operands of the contractions (a few microseconds, timed with the query side)
        const int64_t n4 = (int64_t)(c.num_neg + c.batch) * (c.dim / 4);
        th_split_rows_kernel<<<(int)((n4 + 255) / 256), 256, 0, sq>>>(reinterpret_cast<const float4*>(w.Tneg), c.num_neg,
                                                                     reinterpret_cast<const float4*>(w.What), c.batch, c.dim / 4,
                                                                     reinterpret_cast<uint2*>(w.Tsb), reinterpret_cast<uint2*>(w.Wsb));
        KGE_LAUNCH_CHECK(h);
    }
    KGE_CUDA_CHECK(h, launch_acc_any<true>(p1, tcc, aq, sq));
    stage_end(h, ST_ACCUM_Q, sq);
    KGE_LAUNCH_CHECK(h);
    if (tcc) {
        stage_begin(h, ST_TH_CONTRACT, sq);
        const int rc = launch_th_contract_gemm(h, sq);
        if (rc != KGE_OK) return rc;
        stage_end(h, ST_TH_CONTRACT, sq);
    }
    stage_begin(h, ST_ACCUM_T, st);
    KGE_CUDA_CHECK(h, launch_acc_any<false>(p1, tcc, at, st));
    stage_end(h, ST_ACCUM_T, st);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
