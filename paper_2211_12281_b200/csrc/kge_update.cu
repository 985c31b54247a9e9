// Deterministic de-duplication of touched rows and the sparse row update.
//   rank    : stable sort of the id lists by counting, rank(i) = #{j : (id_j, j) < (id_i, i)}
//   segment : distinct ids, segment offsets (single-CTA scan), batch loss reduction
//   update  : one warp per distinct row: sum the segment's gradient rows in ascending source
//             position, then SGD / Adam / row-wise Adagrad on the table row
#include <cmath>

#include "kge_common.cuh"

namespace kge {

namespace {

struct IdList {
    const int32_t *a, *b, *c;   // the list is the concatenation a[0..na) | b[0..nb) | c[0..nc)
    int na, nb, nc;
    int64_t rows;               // table rows (ids outside [0, rows) are reported and read as 0)
    int32_t *perm, *sorted, *uniq, *seg;
    int32_t* count;             // number of distinct ids
    __device__ __forceinline__ int n() const { return na + nb + nc; }
    __device__ __forceinline__ int32_t raw(int i) const {
        return i < na ? a[i] : (i < na + nb ? b[i - na] : c[i - na - nb]);
    }
};

struct DedupParams {
    IdList ent, rel;
    int ent_blocks;             // rank kernel: blocks [0, ent_blocks) serve the entity list
    int32_t* status;
    const float* Lrow; int B; float loss_scale; float* loss; float* loss_out;
};

constexpr int RANK_THREADS = 256;

__global__ void __launch_bounds__(RANK_THREADS) rank_kernel(DedupParams p) {
    __shared__ int32_t keys[RANK_THREADS];
    const bool is_ent = (int)blockIdx.x < p.ent_blocks;
    const IdList& L = is_ent ? p.ent : p.rel;
    const int n = L.n();
    const int i = (is_ent ? blockIdx.x : blockIdx.x - p.ent_blocks) * RANK_THREADS + threadIdx.x;
    int32_t mine = 0;
    if (i < n) mine = (int32_t)checked_id(L.raw(i), L.rows, p.status);
    int rank = 0;
    for (int j0 = 0; j0 < n; j0 += RANK_THREADS) {
        const int j = j0 + threadIdx.x;
        __syncthreads();
        if (j < n) {
            const int32_t v = L.raw(j);
            keys[threadIdx.x] = (v < 0 || (int64_t)v >= L.rows) ? 0 : v;
        }
        __syncthreads();
        const int m = min(RANK_THREADS, n - j0);
        if (i < n) {
            // positions before i count when id <= mine, positions after i when id < mine
            for (int jj = 0; jj < m; ++jj) {
                const int32_t kj = keys[jj];
                rank += (kj < mine) || (kj == mine && (j0 + jj) < i);
            }
        }
    }
    if (i < n) { L.perm[rank] = i; L.sorted[rank] = mine; }
}

constexpr int SEG_THREADS = 1024;

// blockIdx.x = 0: entity list, 1: relation list, 2: batch loss.
__global__ void __launch_bounds__(SEG_THREADS) segment_kernel(DedupParams p) {
    __shared__ int32_t warp_tot[SEG_THREADS / 32];
    __shared__ int32_t carry;
    __shared__ float lsum[SEG_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (blockIdx.x == 2) {
        float v = 0.f;
        for (int b = tid; b < p.B; b += SEG_THREADS) v += p.Lrow[b];
        v = warp_sum(v);
        if (lane == 0) lsum[warp] = v;
        __syncthreads();
        if (tid == 0) {
            float t = 0.f;
            for (int i = 0; i < SEG_THREADS / 32; ++i) t += lsum[i];
            t *= p.loss_scale;
            *p.loss = t;
            if (p.loss_out) *p.loss_out = t;
        }
        return;
    }
    const IdList& L = blockIdx.x == 0 ? p.ent : p.rel;
    const int n = L.n();
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < n; base += SEG_THREADS) {
        const int r = base + tid;
        const int32_t id = r < n ? L.sorted[r] : 0;
        const int flag = r < n && (r == 0 || L.sorted[r - 1] != id);
        int incl = flag;   // inclusive scan of the head flags
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int before = carry;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (flag) { const int u = before + incl - 1; L.uniq[u] = id; L.seg[u] = r; }
        __syncthreads();
        if (tid == SEG_THREADS - 1) carry = before + incl;
        __syncthreads();
    }
    if (tid == 0) { L.seg[carry] = n; *L.count = carry; }
}

struct UpdateJob {
    float* table; float* state;        // [rows, width], optimiser state
    const float* grads;                // [n, width] gradient rows by source position
    const int32_t *uniq, *seg, *perm;
    const int32_t* count;              // distinct rows (device scalar)
    int width, max_rows;               // max_rows = list length (upper bound of *count)
};

struct UpdateParams {
    UpdateJob job[3];
    int njobs;
    int warp_begin[4];                 // job j serves warps [warp_begin[j], warp_begin[j+1])
    int opt;
    float lr, beta1, beta2, eps, corr1, corr2;   // corr = 1 - beta^t
};

__global__ void __launch_bounds__(256) update_kernel(UpdateParams p) {
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int j = 0;
    while (j + 1 < p.njobs && gw >= p.warp_begin[j + 1]) ++j;
    if (gw >= p.warp_begin[p.njobs]) return;
    const UpdateJob& J = p.job[j];
    const int u = gw - p.warp_begin[j];
    if (u >= *J.count) return;
    const int w4 = J.width >> 2;       // width % 4 == 0 except RotatE relation rows (width % 2 == 0)
    const int64_t row = J.uniq[u];
    const int s0 = J.seg[u], s1 = J.seg[u + 1];
    if ((J.width & 3) == 0) {
        constexpr int MAXC = kMaxDim / 128;
        float4 g[MAXC];
#pragma unroll
        for (int i = 0; i < MAXC; ++i) g[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = s0; s < s1; ++s) {
            const float4* gr = reinterpret_cast<const float4*>(J.grads) + (int64_t)J.perm[s] * w4;
#pragma unroll
            for (int i = 0; i < MAXC; ++i) {
                const int c = lane + 32 * i;
                if (c < w4) { const float4 v = gr[c]; g[i].x += v.x; g[i].y += v.y; g[i].z += v.z; g[i].w += v.w; }
            }
        }
        float4* prow = reinterpret_cast<float4*>(J.table) + row * w4;
        if (p.opt == KGE_OPT_SGD) {
#pragma unroll
            for (int i = 0; i < MAXC; ++i) {
                const int c = lane + 32 * i;
                if (c < w4) {
                    float4 v = prow[c];
                    v.x -= p.lr * g[i].x; v.y -= p.lr * g[i].y; v.z -= p.lr * g[i].z; v.w -= p.lr * g[i].w;
                    prow[c] = v;
                }
            }
        } else if (p.opt == KGE_OPT_ADAM) {
            float4* mrow = reinterpret_cast<float4*>(J.state) + row * 2 * w4;
            float4* vrow = mrow + w4;
#pragma unroll
            for (int i = 0; i < MAXC; ++i) {
                const int c = lane + 32 * i;
                if (c < w4) {
                    float4 m = mrow[c], v = vrow[c], x = prow[c];
                    const float gg[4] = {g[i].x, g[i].y, g[i].z, g[i].w};
                    float* mm = &m.x; float* vv = &v.x; float* xx = &x.x;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        mm[e] = p.beta1 * mm[e] + (1.f - p.beta1) * gg[e];
                        vv[e] = p.beta2 * vv[e] + (1.f - p.beta2) * gg[e] * gg[e];
                        xx[e] -= p.lr * (mm[e] / p.corr1) / (sqrtf(vv[e] / p.corr2) + p.eps);
                    }
                    mrow[c] = m; vrow[c] = v; prow[c] = x;
                }
            }
        } else {
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < MAXC; ++i) ss += g[i].x * g[i].x + g[i].y * g[i].y + g[i].z * g[i].z + g[i].w * g[i].w;
            ss = warp_sum(ss) / (float)J.width;
            const float acc = J.state[row] + ss;
            __syncwarp();
            if (lane == 0) J.state[row] = acc;
            const float step = p.lr / (sqrtf(acc) + p.eps);
#pragma unroll
            for (int i = 0; i < MAXC; ++i) {
                const int c = lane + 32 * i;
                if (c < w4) {
                    float4 v = prow[c];
                    v.x -= step * g[i].x; v.y -= step * g[i].y; v.z -= step * g[i].z; v.w -= step * g[i].w;
                    prow[c] = v;
                }
            }
        }
    } else {
        // narrow rows whose width is only even (RotatE phases with d % 8 != 0): scalar lanes
        constexpr int MAXS = kMaxDim / 2 / 32;
        float g[MAXS];
#pragma unroll
        for (int i = 0; i < MAXS; ++i) g[i] = 0.f;
        for (int s = s0; s < s1; ++s) {
            const float* gr = J.grads + (int64_t)J.perm[s] * J.width;
#pragma unroll
            for (int i = 0; i < MAXS; ++i) { const int c = lane + 32 * i; if (c < J.width) g[i] += gr[c]; }
        }
        float* prow = J.table + row * J.width;
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < MAXS; ++i) ss += g[i] * g[i];
        ss = warp_sum(ss) / (float)J.width;
        float step = p.lr;
        if (p.opt == KGE_OPT_ROWWISE_ADAGRAD) {
            const float acc = J.state[row] + ss;
            __syncwarp();
            if (lane == 0) J.state[row] = acc;
            step = p.lr / (sqrtf(acc) + p.eps);
        }
#pragma unroll
        for (int i = 0; i < MAXS; ++i) {
            const int c = lane + 32 * i;
            if (c >= J.width) continue;
            if (p.opt == KGE_OPT_ADAM) {
                float* m = J.state + row * 2 * J.width + c; float* v = m + J.width;
                const float mm = p.beta1 * *m + (1.f - p.beta1) * g[i];
                const float vv = p.beta2 * *v + (1.f - p.beta2) * g[i] * g[i];
                *m = mm; *v = vv;
                prow[c] -= p.lr * (mm / p.corr1) / (sqrtf(vv / p.corr2) + p.eps);
            } else {
                prow[c] -= step * g[i];
            }
        }
    }
}

}  // namespace

int launch_dedup_update(kge_handle* h, uint64_t step, float lr, const int32_t* heads, const int32_t* rels,
                        const int32_t* tails, const int32_t* negs, float* loss_out, cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg;
    DedupParams dp;
    dp.ent = IdList{heads, tails, negs, B, B, N, c.num_entities, w.ent_perm, w.ent_sorted, w.ent_uniq, w.ent_seg, w.counts};
    dp.rel = IdList{rels, rels, rels, B, 0, 0, c.num_relations, w.rel_perm, w.rel_sorted, w.rel_uniq, w.rel_seg, w.counts + 1};
    dp.ent_blocks = (2 * B + N + RANK_THREADS - 1) / RANK_THREADS;
    dp.status = w.status;
    dp.Lrow = w.Lrow; dp.B = B; dp.loss_scale = c.loss_scale; dp.loss = w.loss; dp.loss_out = loss_out;
    const int rel_blocks = (B + RANK_THREADS - 1) / RANK_THREADS;
    stage_begin(h, ST_RANK, s);
    rank_kernel<<<dp.ent_blocks + rel_blocks, RANK_THREADS, 0, s>>>(dp);
    stage_end(h, ST_RANK, s);
    KGE_LAUNCH_CHECK(h);
    stage_begin(h, ST_SEGMENT, s);
    segment_kernel<<<3, SEG_THREADS, 0, s>>>(dp);
    stage_end(h, ST_SEGMENT, s);
    KGE_LAUNCH_CHECK(h);

    UpdateParams up;
    up.njobs = c.score == KGE_TRANSH ? 3 : 2;
    up.job[0] = UpdateJob{h->ent, h->ent_state, w.grad_ent, w.ent_uniq, w.ent_seg, w.ent_perm, w.counts, c.dim, 2 * B + N};
    up.job[1] = UpdateJob{h->rel, h->rel_state, w.grad_rel, w.rel_uniq, w.rel_seg, w.rel_perm, w.counts + 1, h->kw, B};
    up.job[2] = UpdateJob{h->relw, h->relw_state, w.grad_relw, w.rel_uniq, w.rel_seg, w.rel_perm, w.counts + 1, c.dim, B};
    up.warp_begin[0] = 0;
    for (int j = 0; j < 3; ++j) up.warp_begin[j + 1] = up.warp_begin[j] + (j < up.njobs ? up.job[j].max_rows : 0);
    up.opt = c.opt;
    up.lr = lr; up.beta1 = c.beta1; up.beta2 = c.beta2; up.eps = c.eps;
    up.corr1 = (float)(1.0 - std::pow((double)c.beta1, (double)(step + 1)));
    up.corr2 = (float)(1.0 - std::pow((double)c.beta2, (double)(step + 1)));
    const int warps = up.warp_begin[up.njobs];
    stage_begin(h, ST_UPDATE, s);
    update_kernel<<<(warps * 32 + 255) / 256, 256, 0, s>>>(up);
    stage_end(h, ST_UPDATE, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
