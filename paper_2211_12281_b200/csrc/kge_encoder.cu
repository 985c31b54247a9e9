// Feature-projection encoder (Section 3.1 "Encoder", Eq. 1): e = e_S + M e_F, with M = M_H for heads and M_T for
// tails and negatives.  Around the unchanged scoring step:
//   forward   gather the bf16 feature rows of the batch's 2B + N slots; P = F_slots . M^T on tensor cores (the
//             (B + N) |e_F| d term of the paper's cost model); the gather kernel of the step adds P to the rows it reads
//   backward  the slots' gradient rows (dL/de, which are also the shallow rows' gradients) rounded to bf16;
//             dM_H = dE_heads^T . F_heads, dM_T = dE_tails+negs^T . F_tails+negs as split-K contractions (both operands
//             read MN-major, nothing transposed in memory); one dense optimiser step per matrix that adds the K
//             splits in ascending order
#include <cmath>

#include "kge_common.cuh"

namespace kge {

namespace {

// One warp per slot: the slot's feature row (F bf16 = F / 8 16-byte words).
__global__ void __launch_bounds__(256) feat_gather_kernel(const uint16_t* feat, int F8, int64_t E, const int32_t* heads, const int32_t* tails,
                                                          const int32_t* negs, int B, int N, uint16_t* out, int32_t* status) {
    const int slot = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (slot >= 2 * B + N) return;
    const int32_t raw = slot < B ? heads[slot] : (slot < 2 * B ? tails[slot - B] : negs[slot - 2 * B]);
    const int64_t id = checked_id(raw, E, status);
    const uint4* src = reinterpret_cast<const uint4*>(feat) + id * F8;
    uint4* dst = reinterpret_cast<uint4*>(out) + (int64_t)slot * F8;
    for (int c = lane; c < F8; c += 32) dst[c] = src[c];
}

struct DenseStep {
    float* M; float* state;            // [rows, width]; Adam [rows, 2 width] (m | v); row-wise Adagrad [rows]
    const float* part; int splits;     // [splits][rows, width] partial gradients, added in ascending order
    const float* part2; int splits2;   // a second set (shared matrix: both roles), or NULL
    int rows, width, opt;
    float lr, beta1, beta2, eps, corr1, corr2;
};

// One warp per row of the matrix.
__global__ void __launch_bounds__(256) dense_step_kernel(DenseStep p) {
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (row >= p.rows) return;
    const int64_t slab = (int64_t)p.rows * p.width;
    auto grad = [&](int c) {
        float g = 0.f;
        for (int z = 0; z < p.splits; ++z) g += p.part[z * slab + (int64_t)row * p.width + c];
        if (p.part2) for (int z = 0; z < p.splits2; ++z) g += p.part2[z * slab + (int64_t)row * p.width + c];
        return g;
    };
    float* m = p.M + (int64_t)row * p.width;
    if (p.opt == KGE_OPT_SGD) {
        for (int c = lane; c < p.width; c += 32) m[c] -= p.lr * grad(c);
    } else if (p.opt == KGE_OPT_ADAM) {
        float* m1 = p.state + (int64_t)row * 2 * p.width;
        float* m2 = m1 + p.width;
        for (int c = lane; c < p.width; c += 32) {
            const float g = grad(c);
            const float a = p.beta1 * m1[c] + (1.f - p.beta1) * g, v = p.beta2 * m2[c] + (1.f - p.beta2) * g * g;
            m1[c] = a; m2[c] = v;
            m[c] -= p.lr * (a / p.corr1) / (sqrtf(v / p.corr2) + p.eps);
        }
    } else {
        float ss = 0.f;
        for (int c = lane; c < p.width; c += 32) { const float g = grad(c); ss += g * g; }
        ss = warp_sum(ss) / (float)p.width;
        const float acc = p.state[row] + ss;
        __syncwarp();
        if (lane == 0) p.state[row] = acc;
        const float stepv = p.lr / (sqrtf(acc) + p.eps);
        for (int c = lane; c < p.width; c += 32) m[c] -= stepv * grad(c);
    }
}

}  // namespace

int encoder_make_maps(kge_handle* h) {
    const kge_config& c = h->cfg;
    const Workspace& w = h->ws;
    const int64_t B = c.batch, N = c.num_neg, d = c.dim, F = c.feat_dim;
    int rc = tc_make_operand_map(h, h->tm_fh, w.Fb, B, F, F, 128);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_ft, w.Fb + B * F, B + N, F, F, 128);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_mh, w.Mb, d, F, F, 128);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_mt, w.Mb + d * F, d, F, F, 128);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_gh64, w.Gslot, B, d, d, 64);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_gt64, w.Gslot + B * d, B + N, d, d, 64);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_fh64, w.Fb, B, F, F, 64);
    if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_ft64, w.Fb + B * F, B + N, F, F, 64);
    return rc;
}

int launch_encoder_forward(kge_handle* h, const int32_t* heads, const int32_t* tails, const int32_t* negs, cudaStream_t s) {
    const kge_config& c = h->cfg;
    const Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg, d = c.dim, F = c.feat_dim;
    const int slots = 2 * B + N;
    feat_gather_kernel<<<(slots * 32 + 255) / 256, 256, 0, s>>>(h->feat, F / 8, c.num_entities, heads, tails, negs, B, N, w.Fb, w.status);
    KGE_LAUNCH_CHECK(h);
    int rc = launch_cast_bf16(h, h->MH, w.Mb, (int64_t)d * F, s);
    if (rc == KGE_OK && !c.feat_shared) rc = launch_cast_bf16(h, h->MT, w.Mb + (size_t)d * F, (int64_t)d * F, s);
    if (rc != KGE_OK) return rc;
    const unsigned char* tm_mt = c.feat_shared ? h->tm_mh : h->tm_mt;
    rc = launch_tc_gemm_nt(h, h->tm_fh, h->tm_mh, B, d, F, w.proj, d, s);
    if (rc == KGE_OK) rc = launch_tc_gemm_nt(h, h->tm_ft, tm_mt, B + N, d, F, w.proj + (size_t)B * d, d, s);
    return rc;
}

int launch_encoder_backward(kge_handle* h, uint64_t step, float lr, cudaStream_t s) {
    const kge_config& c = h->cfg;
    const Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg, d = c.dim, F = c.feat_dim;
    int rc = launch_cast_bf16(h, w.grad_ent, w.Gslot, (int64_t)(2 * B + N) * d, s);
    if (rc != KGE_OK) return rc;
    const size_t slab = (size_t)d * F;
    float* partH = w.dMpart;
    float* partT = w.dMpart + (size_t)h->split_m * slab;
    const int splitH = std::min(h->split_m, std::max(1, (B + 63) / 64)), splitT = std::min(h->split_m, std::max(1, (B + N + 63) / 64));
    rc = launch_tc_gemm_tn(h, h->tm_gh64, h->tm_fh64, d, F, B, splitH, partH, F, s);
    if (rc == KGE_OK) rc = launch_tc_gemm_tn(h, h->tm_gt64, h->tm_ft64, d, F, B + N, splitT, partT, F, s);
    if (rc != KGE_OK) return rc;
    auto real_splits = [](int K, int split) { const int kb = (K + 63) / 64, per = (kb + split - 1) / split; return (kb + per - 1) / per; };
    DenseStep p{};
    p.rows = d; p.width = F; p.opt = c.opt;
    p.lr = lr; p.beta1 = c.beta1; p.beta2 = c.beta2; p.eps = c.eps;
    p.corr1 = (float)(1.0 - std::pow((double)c.beta1, (double)(step + 1)));
    p.corr2 = (float)(1.0 - std::pow((double)c.beta2, (double)(step + 1)));
    const int nH = real_splits(B, splitH), nT = real_splits(B + N, splitT);
    const int grid = (d * 32 + 255) / 256;
    if (c.feat_shared) {
        p.M = h->MH; p.state = h->MH_state; p.part = partH; p.splits = nH; p.part2 = partT; p.splits2 = nT;
        dense_step_kernel<<<grid, 256, 0, s>>>(p);
        KGE_LAUNCH_CHECK(h);
    } else {
        p.M = h->MH; p.state = h->MH_state; p.part = partH; p.splits = nH; p.part2 = nullptr; p.splits2 = 0;
        dense_step_kernel<<<grid, 256, 0, s>>>(p);
        KGE_LAUNCH_CHECK(h);
        p.M = h->MT; p.state = h->MT_state; p.part = partT; p.splits = nT;
        dense_step_kernel<<<grid, 256, 0, s>>>(p);
        KGE_LAUNCH_CHECK(h);
    }
    return KGE_OK;
}

}  // namespace kge
