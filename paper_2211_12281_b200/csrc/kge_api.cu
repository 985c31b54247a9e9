// Host side of the C ABI: handle, workspace layout, graph preprocessing, entry points.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "kge_common.cuh"

using namespace kge;

namespace {

// Walks the caller's workspace in 256-byte steps; with base == nullptr it only measures.
struct Carver {
    char* base;
    size_t used = 0;
    explicit Carver(char* b) : base(b) {}
    template <typename T>
    T* take(size_t count) {
        size_t bytes = (count * sizeof(T) + 255) / 256 * 256;
        T* p = base ? reinterpret_cast<T*>(base + used) : nullptr;
        used += bytes;
        return p;
    }
};

int pick_split(int rows, int cols, int num_sms) {
    // One CTA covers 32 owner rows and walks its share of the reduced dimension in chunks of
    // 32; aim for about four CTAs per SM, at most 16 splits, and no empty split.
    const int row_ctas = (rows + 31) / 32;
    const int want = std::max(1, std::min((4 * num_sms + row_ctas / 2) / row_ctas, 16));
    const int per = ((cols + want - 1) / want + 31) / 32 * 32;
    return std::max(1, (cols + per - 1) / per);
}

// The same choice for launches of many more CTAs than the GPU holds at once (TransH at large batches).
int pick_split_waves(int rows, int cols, int num_sms, int ctas_per_sm, int rows_per_cta = 32) {
    // One CTA covers 32 (or 64) owner rows and walks its share of the reduced dimension in chunks of 32.  The CTAs of a launch
    // run in waves of num_sms * ctas_per_sm; the number of column splits (at most 16, none empty) is the one that
    // leaves the last wave fullest, with at least about two waves so that the CTAs' start-up overlaps other CTAs'
    // work, and the fewer splits among equals (every split adds a partial slab for the chain kernel to sum).
    const int row_ctas = (rows + rows_per_cta - 1) / rows_per_cta;
    const int slots = num_sms * ctas_per_sm;
    const int max_split = std::max(1, std::min(16, (cols + 31) / 32));
    int best = 1;
    double best_score = -1.0;
    for (int s = 1; s <= max_split; ++s) {
        const int per = ((cols + s - 1) / s + 31) / 32 * 32;
        const int real = (cols + per - 1) / per;                   // splits that are not empty
        if (real != s) continue;
        const int n = row_ctas * s;
        const int waves = (n + slots - 1) / slots;
        double score = (double)n / ((double)waves * slots);        // how full the waves are
        if (n < 2 * slots) score *= 0.9;                           // fewer than two waves: nothing hides a CTA's start-up
        score -= 0.002 * s;
        if (score > best_score) { best_score = score; best = s; }
    }
    return best;
}

// Tensor-core contraction [rows, cols] over `depth` on persistent CTAs (one per SM): as many K
// splits as still give every SM at most one tile (or one split when there are more tiles than
// SMs), each at least four 64-wide slices deep, at most 16, none empty.
int pick_split_tc(int rows, int cols, int depth, int num_sms) {
    const int bn = tc_backward_tile_cols(cols);
    const int tiles = ((rows + 127) / 128) * ((cols + bn - 1) / bn);
    const int kb = (depth + 63) / 64;
    const int want = std::max(1, std::min(std::min(num_sms / tiles, std::max(1, kb / 4)), 16));
    const int per = (kb + want - 1) / want;
    return (kb + per - 1) / per;
}

size_t layout(const kge_handle* h, char* base, int64_t T, int32_t maxq, int32_t topk, Workspace* out) {
    const kge_config& c = h->cfg;
    const size_t B = c.batch, N = c.num_neg, d = c.dim, kw = h->kw;
    const size_t P = c.num_parts, R = c.num_relations;
    const bool th = c.score == KGE_TRANSH;
    Carver cv(base);
    Workspace w{};
    w.status = cv.take<int32_t>(64);
    w.loss = reinterpret_cast<float*>(w.status ? w.status + 8 : nullptr);
    w.counts = w.status ? w.status + 16 : nullptr;
    w.mrr = reinterpret_cast<double*>(w.status ? w.status + 32 : nullptr);
    w.gh = cv.take<int32_t>(T); w.gr = cv.take<int32_t>(T); w.gt = cv.take<int32_t>(T);
    w.off = cv.take<int64_t>(P * P * (R + 1));
    w.wcum = cv.take<uint64_t>(P * P * (R + 1));
    w.gstart = T > 0 ? cv.take<uint64_t>(P * P * R + 1) : nullptr;
    w.ghist = T > 0 ? cv.take<uint32_t>(graph_hist_words(T)) : nullptr;
    w.heads = cv.take<int32_t>(3 * B + N);
    if (w.heads) { w.rels = w.heads + B; w.tails = w.rels + B; w.negs = w.tails + B; }
    w.Q = cv.take<float>(B * d);
    w.What = th ? cv.take<float>(B * d) : nullptr;
    w.Tneg = cv.take<float>(N * d);
    w.fpos = cv.take<float>(B); w.gpos = cv.take<float>(B); w.Lrow = cv.take<float>(B);
    w.reg_s3 = c.reg_lambda > 0.f ? cv.take<float>(2 * B + N) : nullptr;
    if (c.feat_dim > 0) {
        const size_t F = c.feat_dim;
        w.Fb = cv.take<uint16_t>((2 * B + N) * F);
        w.Mb = cv.take<uint16_t>(2 * d * F);
        w.proj = cv.take<float>((2 * B + N) * d);
        w.Gslot = cv.take<uint16_t>((2 * B + N) * d);
        w.dMpart = cv.take<float>((size_t)2 * h->split_m * d * F);
    }
    const bool tc = c.prec == KGE_PREC_BF16_TC;
    w.Qb = tc ? cv.take<uint16_t>(B * d) : nullptr;
    w.Tb = tc ? cv.take<uint16_t>(N * d) : nullptr;
    w.qn2 = tc ? cv.take<float>(B) : nullptr;
    w.tn2 = tc ? cv.take<float>(N) : nullptr;
    const size_t ldN = (N + 7) / 8 * 8;
    w.Gb = tc ? cv.take<uint16_t>(B * ldN) : nullptr;
    w.Gcol = tc ? cv.take<float>(N) : nullptr;
    const size_t tiles_n = (N + 127) / 128, tiles_m = (B + 127) / 128;
    w.stat_part = tc ? cv.take<float>(B * tc_pieces_per_tile() * tiles_n * 4) : nullptr;
    w.row_stat = tc ? cv.take<float>(B * 2) : nullptr;
    w.grow_part = tc ? cv.take<float>(B * tc_pieces_per_tile() * tiles_n) : nullptr;
    w.gcol_part = tc ? cv.take<float>(4 * tiles_m * N) : nullptr;
    w.Grow = cv.take<float>(B);
    w.Cpart = cv.take<float>((size_t)h->split_t * N);
    w.F = cv.take<float>(B * N);
    w.U = th ? cv.take<float>(B * N) : nullptr;
    w.Cc = th ? cv.take<float>(B * N) : nullptr;
    w.wsum = th ? cv.take<float>(B) : nullptr;
    const size_t Np = (N + 63) / 64 * 64;
    w.Csb = h->th_tc ? cv.take<uint16_t>(B * 2 * Np) : nullptr;
    w.Tsb = h->th_tc ? cv.take<uint16_t>(N * 2 * d) : nullptr;
    w.Wsb = h->th_tc ? cv.take<uint16_t>(B * 2 * d) : nullptr;
    const size_t dp = (d + 63) / 64 * 64;
    w.W3b = h->th_tc ? cv.take<uint16_t>(B * 3 * dp) : nullptr;
    w.T3b = h->th_tc ? cv.take<uint16_t>(N * 3 * dp) : nullptr;
    const size_t xs = (size_t)th_contract_slabs(h);      // slabs the tensor-core contractions add behind the splits' own
    w.dQpart = cv.take<float>((size_t)h->split_q * B * d);
    w.dWpart = th ? cv.take<float>(((size_t)h->split_q + xs) * B * d) : nullptr;
    w.dTpart = cv.take<float>(((size_t)h->split_t + xs) * N * d);
    w.grad_ent = cv.take<float>((2 * B + N) * d);
    w.grad_rel = cv.take<float>(B * kw);
    w.grad_relw = th ? cv.take<float>(B * d) : nullptr;
    const size_t ne = 2 * B + N;
    w.ent_perm = cv.take<int32_t>(ne); w.ent_sorted = cv.take<int32_t>(ne);
    w.ent_uniq = cv.take<int32_t>(ne); w.ent_seg = cv.take<int32_t>(ne + 1);
    w.rel_perm = cv.take<int32_t>(B); w.rel_sorted = cv.take<int32_t>(B);
    w.rel_uniq = cv.take<int32_t>(B); w.rel_seg = cv.take<int32_t>(B + 1);
    w.ent_segof = cv.take<int32_t>(ne); w.rel_segof = cv.take<int32_t>(B);
    w.ent_done = cv.take<int32_t>(ne); w.rel_done = cv.take<int32_t>(B); w.relw_done = th ? cv.take<int32_t>(B) : nullptr;
    w.ent_tkeys = cv.take<uint64_t>((size_t)dedup_tiles((int)ne) * 1024);
    w.rel_tkeys = cv.take<uint64_t>((size_t)dedup_tiles((int)B) * 1024);
    w.part_ent = cv.take<float>(ne * d);
    w.part_rel = cv.take<float>(B * kw);
    w.part_relw = th ? cv.take<float>(B * d) : nullptr;
    if (maxq > 0) {
        const size_t q = maxq, k = std::max(topk, 1);
        w.iq = cv.take<float>(q * d);
        w.iwhat = th ? cv.take<float>(q * d) : nullptr;
        w.iftrue = cv.take<float>(q);
        w.thr = cv.take<float>(q); w.thr_id = cv.take<int32_t>(q);
        w.cand_cnt = cv.take<int32_t>(q); w.beat_tmp = cv.take<int32_t>(q); w.beat = cv.take<int32_t>(q);
        w.cand_score = cv.take<float>(q * kCandCap); w.cand_id = cv.take<int32_t>(q * kCandCap);
        w.top_score = cv.take<float>(q * k); w.top_id = cv.take<int32_t>(q * k);
        w.hq_heads = cv.take<int32_t>(q); w.hq_rels = cv.take<int32_t>(q); w.hq_tails = cv.take<int32_t>(q); w.hq_ranks = cv.take<int32_t>(q);
        w.hq_ids = cv.take<int32_t>(q * k); w.hq_scores = cv.take<float>(q * k);
        // tensor-core inference (dot-product models): bf16 query vectors and a bf16 copy of the whole table
        const bool tci = c.prec == KGE_PREC_BF16_TC && (c.score == KGE_DISTMULT || c.score == KGE_COMPLEX);
        w.iqb = tci ? cv.take<uint16_t>(q * d) : nullptr;
        w.Eb = tci ? cv.take<uint16_t>((size_t)c.num_entities * d) : nullptr;
    }
    if (out) *out = w;
    return cv.used;
}

// Largest w with w^3 <= n * 2^60 (0 for n = 0): integer cube-root sampling weight.
uint64_t icbrt_weight(uint64_t n) {
    if (n == 0) return 0;
    const unsigned __int128 target = (unsigned __int128)n << 60;
    uint64_t lo = 0, hi = (uint64_t)1 << 42;
    while (lo < hi) {
        uint64_t mid = lo + (hi - lo + 1) / 2;
        if ((unsigned __int128)mid * mid * mid <= target) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Mean of (rank <= cutoff ? 1 / rank : 0) over nq ranks in fp64 by one CTA: every thread adds its
// strided share in ascending order, the 256 partial sums are added by a fixed tree, so the result
// is the same on every run.
__global__ void __launch_bounds__(256) mrr_kernel(const int32_t* ranks, int nq, int cutoff, double* out) {
    __shared__ double part[256];
    double acc = 0.0;
    for (int q = threadIdx.x; q < nq; q += 256) {
        const int32_t r = ranks[q];
        if (r >= 1 && (cutoff == 0 || r <= cutoff)) acc += 1.0 / (double)r;
    }
    part[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = part[0] / (double)nq;
}

// One CTA that waits on a barrier nothing ever arrives at: the bounded wait runs out, the kernel
// records KGE_ERR_TIMEOUT and returns.  Exercises the give-up path every kernel of the library shares.
__global__ void wait_probe_kernel(int32_t* status, int limit) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_init_fence(); }
    __syncthreads();
    const bool ok = mbar_wait_bounded(&bar, 0u, limit);
    if (!__syncthreads_and(ok) && threadIdx.x == 0) set_status(status, KGE_ERR_TIMEOUT);
}

}  // namespace

extern "C" {

int kge_create(const kge_config* cfg, kge_handle** out) {
    if (!cfg || !out) return KGE_ERR_BAD_ARG;
    const kge_config& c = *cfg;
    if (c.num_entities <= 0 || c.num_entities > INT32_MAX || c.num_relations <= 0 || c.num_relations > INT32_MAX)
        return KGE_ERR_BAD_ARG;
    if (c.dim <= 0 || c.dim % 4 != 0 || c.dim > kMaxDim) return KGE_ERR_BAD_ARG;
    if (c.score < KGE_TRANSE || c.score > KGE_ROTATE_REAL_L1) return KGE_ERR_BAD_ARG;
    if (c.p_norm != 1 && c.p_norm != 2) return KGE_ERR_BAD_ARG;
    if (c.loss != KGE_LOSS_LOGSIGMOID && c.loss != KGE_LOSS_SAMPLED_SOFTMAX) return KGE_ERR_BAD_ARG;
    if (c.opt < KGE_OPT_SGD || c.opt > KGE_OPT_ROWWISE_ADAGRAD) return KGE_ERR_BAD_ARG;
    if (c.prec != KGE_PREC_FP32 && c.prec != KGE_PREC_BF16_TC) return KGE_ERR_BAD_ARG;
    if (c.batch <= 0 || c.num_neg <= 0 || c.num_parts <= 0) return KGE_ERR_BAD_ARG;
    if (c.head_part >= c.num_parts || c.head_part < -1) return KGE_ERR_BAD_ARG;
    if (c.sample_mode != 0 && c.sample_mode != 1) return KGE_ERR_BAD_ARG;
    if (c.contract < 0 || c.contract > 2) return KGE_ERR_BAD_ARG;
    if (!(c.adv_temp >= 0.f)) return KGE_ERR_BAD_ARG;
    if (!(c.reg_lambda >= 0.f) || (c.reg_form != 0 && c.reg_form != 1)) return KGE_ERR_BAD_ARG;
    if (c.feat_dim < 0 || (c.feat_shared != 0 && c.feat_shared != 1)) return KGE_ERR_BAD_ARG;
    // the projection runs on tensor cores: 64-element slices of the feature axis, 16-byte aligned bf16 rows of width d
    if (c.feat_dim > 0 && (c.feat_dim % 64 != 0 || c.dim % 8 != 0)) return KGE_ERR_UNSUPPORTED;
    if ((int64_t)c.batch * c.num_neg > ((int64_t)1 << 31)) return KGE_ERR_BAD_ARG;
    const int64_t P = c.num_parts;
    if (c.num_neg % P != 0) return KGE_ERR_DIVISIBILITY;
    if (c.head_part < 0 ? (c.batch % (P * P) != 0) : (c.batch % P != 0)) return KGE_ERR_DIVISIBILITY;
    const int64_t S = (c.num_entities + P - 1) / P;
    if (c.num_entities - (P - 1) * S <= 0) return KGE_ERR_EMPTY_BUCKET;  // last partition E_P would be empty
    if (c.prec == KGE_PREC_BF16_TC) {
        // tensor cores serve the scoring functions that are dense contractions: DistMult, ComplEx,
        // and TransE with p = 2 through the norm expansion; rows are cut into 64-element slices
        const bool contraction = c.score == KGE_DISTMULT || c.score == KGE_COMPLEX || (c.score == KGE_TRANSE && c.p_norm == 2);
        if (!contraction || c.dim % 64 != 0) return KGE_ERR_UNSUPPORTED;
    }
    kge_handle* h = new (std::nothrow) kge_handle();
    if (!h) return KGE_ERR_BAD_ARG;
    h->cfg = c;
    h->kind = kind_of(c);
    // RotatE with the real L1 norm differs from RotatE in the pair arithmetic (`kind`) only: from here on it is RotatE
    if (c.score == KGE_ROTATE_REAL_L1) h->cfg.score = KGE_ROTATE;
    h->kw = h->cfg.score == KGE_ROTATE ? c.dim / 2 : c.dim;
    h->bound = h->graph_loaded = false;
    h->streams_ready = false;
    h->launches = 0;
    h->wait_limit = kDefaultWaitLimit;
    h->capture_scores = nullptr;
    h->cuda_err[0] = '\0';
    h->num_sms = 148;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
        h->num_sms = sms;
    else
        (void)cudaGetLastError();
    // TransH, fp32: its three dense contractions (u = w.t; the backward's two sums with one coefficient per pair) go
    // to the tensor cores as bf16 splits once a block has enough pairs to pay for the extra launches (`contract`:
    // 0 automatic, 1 always where the shapes allow, 2 never)
    h->th_tc = c.score == KGE_TRANSH && c.prec == KGE_PREC_FP32 && c.dim % 32 == 0 && c.contract != 2 &&
               (c.contract == 1 || (int64_t)c.batch * c.num_neg >= ((int64_t)1 << 22));
    // resident CTAs per SM of the TransH accumulation kernels: two (128 registers x 256 threads, 70-90 KB of shared memory);
    // with the c sums on the tensor cores a CTA of the negatives' side owns 64 rows
    if (c.score == KGE_TRANSH) {
        h->split_q = pick_split_waves(c.batch, c.num_neg, h->num_sms, 2);
        h->split_t = pick_split_waves(c.num_neg, c.batch, h->num_sms, 2, h->th_tc ? 64 : 32);
    } else {
        h->split_q = pick_split(c.batch, c.num_neg, h->num_sms);
        h->split_t = pick_split(c.num_neg, c.batch, h->num_sms);
    }
    if (c.prec == KGE_PREC_BF16_TC) {   // the backward contractions run as 128 x 128 tensor-core tiles split over K
        h->split_q = pick_split_tc(c.batch, c.dim, c.num_neg, h->num_sms);
        h->split_t = pick_split_tc(c.num_neg, c.dim, c.batch, h->num_sms);
    }
    h->th_gsplit = 1;
    if (h->th_tc) {   // K splits: as many as still give every SM at most one tile, each at least eight 64-wide slices deep, at most 4
        const int bn = 2 * c.dim > 128 ? 256 : 128;
        const int tiles = ((c.batch + 127) / 128 + (c.num_neg + 127) / 128) * ((2 * c.dim + bn - 1) / bn);
        const int kb = 2 * ((std::min(c.batch, c.num_neg) + 63) / 64);
        h->th_gsplit = std::max(1, std::min(std::min(h->num_sms / tiles, kb / 8), 4));
    }
    h->split_m = 1;
    h->features_bound = false;
    if (c.feat_dim > 0)   // dM = dE^T . F: [d, F] over the batch's slots, split over the slots so that every SM has a tile
        h->split_m = pick_split_tc(c.dim, c.feat_dim, c.batch, h->num_sms);
    *out = h;
    return KGE_OK;
}

void kge_destroy(kge_handle* h) {
    if (!h) return;
    if (h->prof.created)
        for (int i = 0; i < ST_COUNT; ++i) { cudaEventDestroy(h->prof.a[i]); cudaEventDestroy(h->prof.b[i]); }
    if (h->streams_ready) {
        cudaStreamDestroy(h->side[0]); cudaStreamDestroy(h->side[1]);
        cudaEventDestroy(h->ev_ids); cudaEventDestroy(h->ev_loss); cudaEventDestroy(h->ev_seg); cudaEventDestroy(h->ev_t);
    }
    delete h;
}

int kge_profile(kge_handle* h, int enable) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (enable && !h->prof.created) {
        for (int i = 0; i < ST_COUNT; ++i) {
            KGE_CUDA_CHECK(h, cudaEventCreate(&h->prof.a[i]));
            KGE_CUDA_CHECK(h, cudaEventCreate(&h->prof.b[i]));
        }
        h->prof.created = true;
    }
    h->prof.on = enable != 0;
    return KGE_OK;
}

int kge_profile_read(kge_handle* h, double* ms, int64_t* launches, int reset) {
    if (!h || !ms || !launches) return KGE_ERR_BAD_ARG;
    for (int i = 0; i < ST_COUNT; ++i) {
        ms[i] = h->prof.ms[i]; launches[i] = h->prof.n[i];
        if (reset) { h->prof.ms[i] = 0.0; h->prof.n[i] = 0; }
    }
    return KGE_OK;
}

size_t kge_workspace_bytes(const kge_handle* h, int64_t num_triples, int32_t max_queries, int32_t topk) {
    if (!h || num_triples < 0 || max_queries < 0 || topk < 0) return 0;
    return layout(h, nullptr, num_triples, max_queries, topk, nullptr);
}

int kge_bind(kge_handle* h, float* ent, float* rel, float* relw, float* ent_state, float* rel_state,
             float* relw_state, void* workspace, size_t workspace_bytes, int64_t num_triples,
             int32_t max_queries, int32_t topk, void* stream) {
    if (!h || !ent || !rel) return KGE_ERR_BAD_ARG;
    if (h->cfg.score == KGE_TRANSH && !relw) return KGE_ERR_BAD_ARG;
    if (h->cfg.opt != KGE_OPT_SGD && (!ent_state || !rel_state || (h->cfg.score == KGE_TRANSH && !relw_state)))
        return KGE_ERR_BAD_ARG;
    if (num_triples < 0 || max_queries < 0 || topk < 0 || topk > kCandCap) return KGE_ERR_BAD_ARG;
    auto misaligned = [](const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) != 0; };
    if (misaligned(ent, 16) || misaligned(rel, 16) || misaligned(relw, 16) || misaligned(ent_state, 16) ||
        misaligned(rel_state, 16) || misaligned(relw_state, 16) || misaligned(workspace, 256))
        return KGE_ERR_BAD_ARG;
    if (!workspace || workspace_bytes < layout(h, nullptr, num_triples, max_queries, topk, nullptr))
        return KGE_ERR_WORKSPACE;
    h->ent = ent; h->rel = rel; h->relw = relw;
    h->ent_state = ent_state; h->rel_state = rel_state; h->relw_state = relw_state;
    h->ws_base = static_cast<char*>(workspace);
    h->ws_bytes = workspace_bytes;
    h->num_triples = num_triples; h->max_queries = max_queries; h->topk = topk;
    h->tiles32_ready = false;       // (tensor maps of the inference tiles are encoded at the first full-entity call)
    layout(h, h->ws_base, num_triples, max_queries, topk, &h->ws);
    KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.status, 0, 256, static_cast<cudaStream_t>(stream)));
    if (h->cfg.prec == KGE_PREC_BF16_TC) {
        const int64_t B = h->cfg.batch, N = h->cfg.num_neg, d = h->cfg.dim;
        const int64_t ldN = (N + 7) / 8 * 8;
        int rc = tc_make_operand_map(h, h->tm_q, h->ws.Qb, B, d, d, 128);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_t, h->ws.Tb, N, d, d, 128);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_g, h->ws.Gb, B, N, ldN, 128);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_g64, h->ws.Gb, B, N, ldN, 64);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_t64, h->ws.Tb, N, d, d, 64);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_q64, h->ws.Qb, B, d, d, 64);
        if (rc == KGE_OK && h->ws.Eb) {
            rc = tc_make_operand_map(h, h->tm_iq, h->ws.iqb, max_queries, d, d, 128);
            if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_eb, h->ws.Eb, h->cfg.num_entities, d, d, 128);
        }
        if (rc != KGE_OK) return rc;
    }
    if (h->th_tc) {
        const int64_t B = h->cfg.batch, N = h->cfg.num_neg, d = h->cfg.dim, Np = (N + 63) / 64 * 64;
        // (the padding columns of the coefficient splits are never written: zero once, zero for good)
        KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.Csb, 0, (size_t)B * 2 * Np * 2, static_cast<cudaStream_t>(stream)));
        int rc = tc_make_operand_map(h, h->tm_cs, h->ws.Csb, B, 2 * Np, 2 * Np, 128);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_cs64, h->ws.Csb, B, 2 * Np, 2 * Np, 64);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_ts64, h->ws.Tsb, N, 2 * d, 2 * d, 64);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_ws64, h->ws.Wsb, B, 2 * d, 2 * d, 64);
        const int64_t dp = (d + 63) / 64 * 64;
        KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.W3b, 0, (size_t)B * 3 * dp * 2, static_cast<cudaStream_t>(stream)));
        KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.T3b, 0, (size_t)N * 3 * dp * 2, static_cast<cudaStream_t>(stream)));
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_w3, h->ws.W3b, B, 3 * dp, 3 * dp, 128);
        if (rc == KGE_OK) rc = tc_make_operand_map(h, h->tm_t3, h->ws.T3b, N, 3 * dp, 3 * dp, 128);
        if (rc != KGE_OK) return rc;
    }
    if (!h->streams_ready) {
        // side[0] carries the sort of the touched ids, a few small kernels the update waits for:
        // at the highest priority their CTAs take the next free slots instead of queueing behind
        // the score and gradient kernels' hundreds of CTAs
        int prio_least = 0, prio_greatest = 0;
        KGE_CUDA_CHECK(h, cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
        KGE_CUDA_CHECK(h, cudaStreamCreateWithPriority(&h->side[0], cudaStreamNonBlocking, prio_greatest));
        KGE_CUDA_CHECK(h, cudaStreamCreateWithFlags(&h->side[1], cudaStreamNonBlocking));
        cudaEvent_t* evs[4] = {&h->ev_ids, &h->ev_loss, &h->ev_seg, &h->ev_t};
        for (cudaEvent_t* e : evs) KGE_CUDA_CHECK(h, cudaEventCreateWithFlags(e, cudaEventDisableTiming));
        h->streams_ready = true;
    }
    h->bound = true;
    h->graph_loaded = false;
    h->eb_valid = false;
    return KGE_OK;
}

int kge_bind_features(kge_handle* h, const uint16_t* feat, float* MH, float* MT, float* MH_state, float* MT_state, void* stream) {
    (void)stream;
    if (!h || !feat || !MH || !MT) return KGE_ERR_BAD_ARG;
    if (h->cfg.feat_dim <= 0) return KGE_ERR_UNSUPPORTED;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if ((h->cfg.feat_shared != 0) != (MH == MT)) return KGE_ERR_BAD_ARG;
    if (h->cfg.opt != KGE_OPT_SGD && (!MH_state || !MT_state)) return KGE_ERR_BAD_ARG;
    auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) % 16) != 0; };
    if (misaligned(feat) || misaligned(MH) || misaligned(MT)) return KGE_ERR_BAD_ARG;
    h->feat = feat; h->MH = MH; h->MT = MT; h->MH_state = MH_state; h->MT_state = MT_state;
    const int rc = encoder_make_maps(h);
    if (rc != KGE_OK) return rc;
    h->features_bound = true;
    return KGE_OK;
}

int kge_graph_load(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails, int64_t n,
                   void* stream) {
    if (!h || !heads || !rels || !tails || n < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (n != h->num_triples) return KGE_ERR_WORKSPACE;
    const kge_config& c = h->cfg;
    const int64_t E = c.num_entities, R = c.num_relations, P = c.num_parts;
    const int64_t S = (E + P - 1) / P;
    const int64_t nkeys = P * P * R;
    std::vector<int64_t> start(nkeys + 1, 0);
    for (int64_t e = 0; e < n; ++e) {
        if (heads[e] < 0 || heads[e] >= E || tails[e] < 0 || tails[e] >= E || rels[e] < 0 || rels[e] >= R)
            return KGE_ERR_BAD_ARG;
        start[((heads[e] / S) * P + tails[e] / S) * R + rels[e] + 1] += 1;
    }
    for (int64_t k = 0; k < nkeys; ++k) start[k + 1] += start[k];
    std::vector<int64_t> off(P * P * (R + 1));
    std::vector<uint64_t> wcum(P * P * (R + 1));
    for (int64_t b = 0; b < P * P; ++b) {
        uint64_t acc = 0;
        for (int64_t r = 0; r <= R; ++r) {
            off[b * (R + 1) + r] = start[b * R + r];
            wcum[b * (R + 1) + r] = acc;
            if (r < R) acc += icbrt_weight((uint64_t)(start[b * R + r + 1] - start[b * R + r]));
        }
        const bool needed = c.head_part < 0 || b / P == c.head_part;
        const bool empty = c.sample_mode == 0 ? acc == 0 : start[b * R + R] == start[b * R];
        if (needed && empty) return KGE_ERR_EMPTY_BUCKET;
    }
    std::vector<int32_t> sh(n), sr(n), st(n);
    std::vector<int64_t> cursor(start.begin(), start.end() - 1);
    for (int64_t e = 0; e < n; ++e) {  // input order inside a key is kept: stable
        int64_t dst = cursor[((heads[e] / S) * P + tails[e] / S) * R + rels[e]]++;
        sh[dst] = heads[e]; sr[dst] = rels[e]; st[dst] = tails[e];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace& w = h->ws;
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.gh, sh.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.gr, sr.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.gt, st.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.off, off.data(), off.size() * sizeof(int64_t), cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.wcum, wcum.data(), wcum.size() * sizeof(uint64_t), cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    h->graph_loaded = true;
    return KGE_OK;
}

int kge_graph_load_device(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails, int64_t n,
                          void* stream) {
    if (!h || !heads || !rels || !tails || n < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (n != h->num_triples) return KGE_ERR_WORKSPACE;
    const kge_config& c = h->cfg;
    // keys and triple indices are sorted as 32-bit words
    if (n > ((int64_t)1 << 31) || (int64_t)c.num_parts * c.num_parts * c.num_relations > ((int64_t)1 << 31)) return KGE_ERR_UNSUPPORTED;
    h->graph_loaded = false;
    if (n == 0) return KGE_ERR_EMPTY_BUCKET;      // every bucket is empty
    const int rc = launch_graph_build_device(h, heads, rels, tails, n, static_cast<cudaStream_t>(stream));
    if (rc != KGE_OK) return rc;
    h->graph_loaded = true;
    return KGE_OK;
}

int kge_init_tables(kge_handle* h, float std, void* stream) {
    if (!h || !(std >= 0.f)) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    const kge_config& c = h->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    h->eb_valid = false;
    int rc = launch_init_table(h, h->ent, c.num_entities, c.dim, std, 0, 2u, s);
    if (rc == KGE_OK) rc = launch_init_table(h, h->rel, c.num_relations, h->kw, std, c.score == KGE_ROTATE ? 1 : 0, 3u, s);
    if (rc == KGE_OK && h->relw) rc = launch_init_table(h, h->relw, c.num_relations, c.dim, std, 0, 4u, s);
    if (rc != KGE_OK) return rc;
    // optimiser state starts at zero
    const size_t per = c.opt == KGE_OPT_ADAM ? 2 : 1;
    if (c.opt != KGE_OPT_SGD) {
        const bool adam = c.opt == KGE_OPT_ADAM;
        KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ent_state, 0, (size_t)c.num_entities * (adam ? per * c.dim : 1) * sizeof(float), s));
        KGE_CUDA_CHECK(h, cudaMemsetAsync(h->rel_state, 0, (size_t)c.num_relations * (adam ? per * h->kw : 1) * sizeof(float), s));
        if (h->relw_state)
            KGE_CUDA_CHECK(h, cudaMemsetAsync(h->relw_state, 0, (size_t)c.num_relations * (adam ? per * c.dim : 1) * sizeof(float), s));
    }
    return KGE_OK;
}

int kge_debug_init_words(kge_handle* h, float* out, int64_t rows, int32_t width, uint32_t stream_id, void* stream) {
    if (!h || !out || rows < 0 || width <= 0) return KGE_ERR_BAD_ARG;
    return launch_init_table(h, out, rows, width, 1.f, 2, stream_id, static_cast<cudaStream_t>(stream));
}

int kge_sample_batch(kge_handle* h, uint64_t step, int32_t* heads, int32_t* rels, int32_t* tails, int32_t* negs,
                     void* stream) {
    if (!h || !heads || !rels || !tails || !negs) return KGE_ERR_BAD_ARG;
    if (!h->bound || !h->graph_loaded) return KGE_ERR_NOT_READY;
    return launch_sample(h, step, heads, rels, tails, negs, static_cast<cudaStream_t>(stream));
}

int kge_train_step(kge_handle* h, uint64_t step, float lr, const int32_t* heads, const int32_t* rels,
                   const int32_t* tails, const int32_t* negs, float* loss_out, void* stream) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    const int given = (heads != nullptr) + (rels != nullptr) + (tails != nullptr) + (negs != nullptr);
    if (given != 0 && given != 4) return KGE_ERR_BAD_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace& w = h->ws;
    // With per-stage timing on, everything runs in order on the caller's stream.  Otherwise
    // the sort of the touched ids (which needs only the ids) runs on a side stream beside
    // the forward and backward kernels, and joins before the update.
    const bool fork = !h->prof.on;
    bool fused = false;
    int rc;
    if (given == 0) {
        if (!h->graph_loaded) return KGE_ERR_NOT_READY;
        // The gather kernel can draw the batch itself when the 8 query warps of a CTA share a
        // triple bucket and the bucket's cumulative weights fit its shared memory.
        const kge_config& c = h->cfg;
        const int buckets = c.head_part < 0 ? c.num_parts * c.num_parts : c.num_parts;
        // (with an encoder the ids must exist before the gather: the features of the batch are projected first)
        fused = fork && (c.batch / buckets) % 8 == 0 && c.num_relations + 1 <= 4096 && c.feat_dim == 0;
        if (!fused) {
            rc = launch_sample(h, step, w.heads, w.rels, w.tails, w.negs, s);
            if (rc != KGE_OK) return rc;
        }
        heads = w.heads; rels = w.rels; tails = w.tails; negs = w.negs;
    }
    if (h->cfg.feat_dim > 0) {
        if (!h->features_bound) return KGE_ERR_NOT_READY;
        if ((rc = launch_encoder_forward(h, heads, tails, negs, s)) != KGE_OK) return rc;
    }
    rc = launch_forward_backward(h, heads, rels, tails, negs, loss_out, s, fork ? h->side[1] : nullptr,
                                 fork ? h->side[0] : nullptr, fused, step);
    if (rc != KGE_OK) return rc;
    // with side streams the id sort has been joined before the chain kernel
    if (!fork && (rc = launch_dedup(h, heads, rels, tails, negs, s)) != KGE_OK) return rc;
    rc = launch_update(h, step, lr, s);
    if (rc == KGE_OK && h->cfg.feat_dim > 0) rc = launch_encoder_backward(h, step, lr, s);
    h->eb_valid = false;          // the entity table has moved on: tensor-core inference must refresh its bf16 copy
    if (rc != KGE_OK) return rc;
    return h->prof.on ? stage_collect(h, s) : KGE_OK;
}

int kge_train_gradients(kge_handle* h, uint64_t step, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                        const int32_t* negs, float* loss_out, void* stream) {
    if (!h || !heads || !rels || !tails || !negs) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (h->cfg.feat_dim > 0) return KGE_ERR_UNSUPPORTED;
    // forward and backward only, in order on the caller's stream: no sort of the touched ids, no update
    return launch_forward_backward(h, heads, rels, tails, negs, loss_out, static_cast<cudaStream_t>(stream), nullptr, nullptr, false, step);
}

int kge_gradient_rows(kge_handle* h, float** grad_ent, float** grad_rel, float** grad_relw) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (grad_ent) *grad_ent = h->ws.grad_ent;
    if (grad_rel) *grad_rel = h->ws.grad_rel;
    if (grad_relw) *grad_relw = h->ws.grad_relw;
    return KGE_OK;
}

int kge_gather_rows(kge_handle* h, const int32_t* ids, int32_t n, int64_t ent_base, float* rows_out, void* stream) {
    if (!h || !ids || !rows_out || n < 0 || ent_base < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (n == 0) return KGE_OK;
    return launch_gather_rows(h, ids, n, ent_base, rows_out, static_cast<cudaStream_t>(stream));
}

size_t kge_apply_scratch_bytes(const kge_handle* h, int32_t table, int32_t n) {
    if (!h || n <= 0 || table < 0 || table > 2) return 0;
    return apply_scratch_bytes(n, table == 1 ? h->kw : h->cfg.dim);
}

int kge_apply_gradients(kge_handle* h, int32_t table, const int32_t* ids, const float* grads, int32_t n, uint64_t step, float lr,
                        void* scratch, size_t scratch_bytes, void* stream) {
    if (!h || !ids || !grads || n < 0 || table < 0 || table > 2) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (n == 0) return KGE_OK;
    float* tab = table == 0 ? h->ent : (table == 1 ? h->rel : h->relw);
    float* state = table == 0 ? h->ent_state : (table == 1 ? h->rel_state : h->relw_state);
    if (!tab) return KGE_ERR_BAD_ARG;
    const int width = table == 1 ? h->kw : h->cfg.dim;
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) % 256) != 0 || scratch_bytes < apply_scratch_bytes(n, width)) return KGE_ERR_WORKSPACE;
    const int64_t rows = table == 0 ? h->cfg.num_entities : h->cfg.num_relations;
    h->eb_valid = false;
    return launch_apply_gradients(h, tab, state, rows, width, ids, grads, n, step, lr, scratch, static_cast<cudaStream_t>(stream));
}

int kge_train_step_host(kge_handle* h, uint64_t step, float lr, const int32_t* heads, const int32_t* rels,
                        const int32_t* tails, const int32_t* negs, float* loss_out, void* stream) {
    if (!h || !heads || !rels || !tails || !negs) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace& w = h->ws;
    const size_t B = h->cfg.batch, N = h->cfg.num_neg;
    if (rels == heads + B && tails == rels + B && negs == tails + B) {
        // the four lists lie back to back on the host, as they do in the workspace: one copy
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.heads, heads, (3 * B + N) * 4, cudaMemcpyHostToDevice, s));
    } else {
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.heads, heads, B * 4, cudaMemcpyHostToDevice, s));
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.rels, rels, B * 4, cudaMemcpyHostToDevice, s));
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.tails, tails, B * 4, cudaMemcpyHostToDevice, s));
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.negs, negs, N * 4, cudaMemcpyHostToDevice, s));
    }
    int rc = kge_train_step(h, step, lr, w.heads, w.rels, w.tails, w.negs, w.loss, stream);
    if (rc != KGE_OK) return rc;
    if (loss_out) KGE_CUDA_CHECK(h, cudaMemcpyAsync(loss_out, w.loss, 4, cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return KGE_OK;
}

int kge_score_all_topk(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int32_t k,
                       const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                       void* stream) {
    if (!h || nq < 0 || k <= 0) return KGE_ERR_BAD_ARG;
    if (nq > 0 && (!q_heads || !q_rels || !out_ids || !out_scores)) return KGE_ERR_BAD_ARG;   // an empty batch may pass NULL
    if (out_ranks && !true_tails) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (h->cfg.feat_dim > 0) return KGE_ERR_UNSUPPORTED;      // full-entity scoring reads shallow rows only
    if (nq > h->max_queries || k > h->topk) return KGE_ERR_WORKSPACE;
    if (nq == 0) return KGE_OK;
    return run_score_all_topk(h, q_heads, q_rels, nq, k, true_tails, out_ids, out_scores, out_ranks,
                              static_cast<cudaStream_t>(stream));
}

int kge_score_all_topk_host(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int32_t k,
                            const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                            void* stream) {
    if (!h || nq < 0 || k <= 0) return KGE_ERR_BAD_ARG;
    if (nq > 0 && (!q_heads || !q_rels || !out_ids || !out_scores)) return KGE_ERR_BAD_ARG;
    if (out_ranks && !true_tails) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (nq > h->max_queries || k > h->topk) return KGE_ERR_WORKSPACE;
    if (nq == 0) return KGE_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Workspace& w = h->ws;
    const size_t qb = (size_t)nq * sizeof(int32_t);
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.hq_heads, q_heads, qb, cudaMemcpyHostToDevice, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.hq_rels, q_rels, qb, cudaMemcpyHostToDevice, s));
    if (true_tails) KGE_CUDA_CHECK(h, cudaMemcpyAsync(w.hq_tails, true_tails, qb, cudaMemcpyHostToDevice, s));
    const int rc = run_score_all_topk(h, w.hq_heads, w.hq_rels, nq, k, true_tails ? w.hq_tails : nullptr, w.hq_ids, w.hq_scores,
                                      out_ranks ? w.hq_ranks : nullptr, s);
    if (rc != KGE_OK) return rc;
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(out_ids, w.hq_ids, (size_t)nq * k * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(out_scores, w.hq_scores, (size_t)nq * k * sizeof(float), cudaMemcpyDeviceToHost, s));
    if (out_ranks) KGE_CUDA_CHECK(h, cudaMemcpyAsync(out_ranks, w.hq_ranks, qb, cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return KGE_OK;
}

int kge_shard_query_vectors(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int64_t ent_base,
                            float* qvec_out, void* stream) {
    if (!h || !q_heads || !q_rels || !qvec_out || nq <= 0 || ent_base < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (nq > h->max_queries) return KGE_ERR_WORKSPACE;
    return run_shard_query_vectors(h, q_heads, q_rels, nq, ent_base, qvec_out, static_cast<cudaStream_t>(stream));
}

int kge_shard_true_scores(kge_handle* h, const float* qvec, const int32_t* q_rels, const int32_t* true_tails, int32_t nq,
                          int64_t ent_base, float* ftrue_out, void* stream) {
    if (!h || !qvec || !q_rels || !true_tails || !ftrue_out || nq <= 0 || ent_base < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (nq > h->max_queries) return KGE_ERR_WORKSPACE;
    return run_shard_true_scores(h, qvec, q_rels, true_tails, nq, ent_base, ftrue_out, static_cast<cudaStream_t>(stream));
}

int kge_shard_score_topk(kge_handle* h, const float* qvec, const int32_t* q_rels, int32_t nq, int32_t k, const float* ftrue,
                         const int32_t* true_tails, int64_t ent_base, int32_t* out_ids, float* out_scores, int32_t* out_beat,
                         void* stream) {
    if (!h || !qvec || !q_rels || !out_ids || !out_scores || nq <= 0 || k <= 0 || ent_base < 0) return KGE_ERR_BAD_ARG;
    if ((out_beat != nullptr) != (true_tails != nullptr) || (true_tails != nullptr) != (ftrue != nullptr)) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (nq > h->max_queries || k > h->topk) return KGE_ERR_WORKSPACE;
    if (ent_base + h->cfg.num_entities > INT32_MAX) return KGE_ERR_BAD_ARG;     // ids stay 32-bit
    const ShardScoring shard{ent_base, qvec, ftrue};
    return run_score_all_topk(h, nullptr, q_rels, nq, k, true_tails, out_ids, out_scores, out_beat, static_cast<cudaStream_t>(stream), &shard);
}

int kge_merge_topk(const int32_t* cand_ids, const float* cand_scores, int32_t nq, int32_t per_query, int32_t k, int32_t* out_ids,
                   float* out_scores, void* stream) {
    if (!cand_ids || !cand_scores || !out_ids || !out_scores || nq < 0 || per_query <= 0 || k <= 0) return KGE_ERR_BAD_ARG;
    if (nq == 0) return KGE_OK;
    return run_merge_topk(cand_ids, cand_scores, nq, per_query, k, out_ids, out_scores, static_cast<cudaStream_t>(stream));
}

int kge_refresh_inference_table(kge_handle* h, void* stream) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (!h->ws.Eb) return KGE_OK;
    const int rc = launch_cast_bf16(h, h->ent, h->ws.Eb, h->cfg.num_entities * h->cfg.dim, static_cast<cudaStream_t>(stream));
    if (rc == KGE_OK) h->eb_valid = true;
    return rc;
}

int kge_mrr_from_ranks(kge_handle* h, const int32_t* ranks, int32_t nq, int32_t k_cutoff, double* mrr_out, void* stream) {
    if (!h || !ranks || !mrr_out || nq <= 0 || k_cutoff < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    mrr_kernel<<<1, 256, 0, s>>>(ranks, nq, k_cutoff, h->ws.mrr);
    KGE_LAUNCH_CHECK(h);
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(mrr_out, h->ws.mrr, sizeof(double), cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return KGE_OK;
}

int kge_eval_mrr(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, const int32_t* true_tails,
                 int32_t nq, int32_t k_cutoff, double* mrr_out, void* stream) {
    if (!h || !q_heads || !q_rels || !true_tails || !mrr_out || nq <= 0 || k_cutoff < 0) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    if (nq > h->max_queries || h->topk < 1) return KGE_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a k = 1 search whose lists are discarded; only the ranks are used (they land in the workspace)
    const int rc = run_score_all_topk(h, q_heads, q_rels, nq, 1, true_tails, nullptr, nullptr, h->ws.beat_tmp, s);
    if (rc != KGE_OK) return rc;
    return kge_mrr_from_ranks(h, h->ws.beat_tmp, nq, k_cutoff, mrr_out, stream);
}

int kge_debug_set_wait_limit(kge_handle* h, int32_t tries) {
    if (!h || tries < 0) return KGE_ERR_BAD_ARG;
    h->wait_limit = tries == 0 ? kDefaultWaitLimit : tries;
    return KGE_OK;
}

int kge_debug_wait_probe(kge_handle* h, void* stream) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    wait_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(h->ws.status, h->wait_limit);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

int kge_debug_capture_scores(kge_handle* h, float* scores_out) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (scores_out && (reinterpret_cast<uintptr_t>(scores_out) % 16) != 0) return KGE_ERR_BAD_ARG;
    h->capture_scores = scores_out;
    return KGE_OK;
}

float kge_lr_linear_decay(float lr0, uint64_t step, uint64_t total_steps) {
    if (total_steps == 0 || step >= total_steps) return 0.f;
    return (float)((double)lr0 * (1.0 - (double)step / (double)total_steps));
}

int kge_get_status(kge_handle* h, void* stream) {
    if (!h) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(&word, h->ws.status, 4, cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaMemsetAsync(h->ws.status, 0, 4, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return word;
}

}  // extern "C"

namespace kge {
int stage_collect(kge_handle* h, cudaStream_t s) {
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    for (int i = 0; i < ST_COUNT; ++i) {
        if (!h->prof.used[i]) continue;
        float ms = 0.f;
        KGE_CUDA_CHECK(h, cudaEventElapsedTime(&ms, h->prof.a[i], h->prof.b[i]));
        h->prof.ms[i] += ms; h->prof.n[i] += 1; h->prof.used[i] = false;
    }
    return KGE_OK;
}
}  // namespace kge

extern "C" {

int64_t kge_launch_count(const kge_handle* h) { return h ? h->launches : 0; }

const char* kge_error_string(int code) {
    switch (code) {
        case KGE_OK: return "ok";
        case KGE_ERR_BAD_ARG: return "bad argument";
        case KGE_ERR_DIVISIBILITY: return "batch / negatives not divisible by the partition count";
        case KGE_ERR_EMPTY_BUCKET: return "a triple bucket or entity partition that must be sampled is empty";
        case KGE_ERR_WORKSPACE: return "workspace missing, too small, or sized for other limits";
        case KGE_ERR_UNSUPPORTED: return "combination not implemented";
        case KGE_ERR_NOT_READY: return "tables not bound or graph not loaded";
        case KGE_ERR_CUDA: return "CUDA runtime error";
        case KGE_ERR_ID_RANGE: return "an entity or relation id was outside its table";
        case KGE_ERR_TOPK_OVERFLOW: return "top-k candidate list overflow";
        case KGE_ERR_NO_EXTENSION: return "CUDA extension not built";
        case KGE_ERR_TIMEOUT: return "a bounded wait on an asynchronous copy ran out";
        default: return "unknown error";
    }
}

const char* kge_last_cuda_error(const kge_handle* h) { return h ? h->cuda_err : ""; }

size_t kge_debug_bytes(kge_handle* h, int tap, void* stream) {
    if (!h || !h->bound) return 0;
    const kge_config& c = h->cfg;
    const size_t B = c.batch, N = c.num_neg, d = c.dim;
    int32_t counts[2] = {0, 0};
    if (tap == KGE_TAP_ENT_UNIQ || tap == KGE_TAP_ENT_SEG || tap == KGE_TAP_REL_UNIQ || tap == KGE_TAP_REL_SEG) {
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        if (cudaMemcpyAsync(counts, h->ws.counts, 8, cudaMemcpyDeviceToHost, s) != cudaSuccess) return 0;
        if (cudaStreamSynchronize(s) != cudaSuccess) return 0;
    }
    switch (tap) {
        case KGE_TAP_Q: return B * d * 4;
        case KGE_TAP_FPOS: case KGE_TAP_LROW: return B * 4;
        case KGE_TAP_G: return B * N * 4;
        case KGE_TAP_GRAD_ENT: return (2 * B + N) * d * 4;
        case KGE_TAP_GRAD_REL: return B * h->kw * 4;
        case KGE_TAP_GRAD_RELW: return c.score == KGE_TRANSH ? B * d * 4 : 0;
        case KGE_TAP_ENT_UNIQ: return (size_t)counts[0] * 4;
        case KGE_TAP_ENT_SEG: return ((size_t)counts[0] + 1) * 4;
        case KGE_TAP_ENT_PERM: return (2 * B + N) * 4;
        case KGE_TAP_REL_UNIQ: return (size_t)counts[1] * 4;
        case KGE_TAP_REL_SEG: return ((size_t)counts[1] + 1) * 4;
        case KGE_TAP_REL_PERM: return B * 4;
        case KGE_TAP_BATCH: return (3 * B + N) * 4;
        case KGE_TAP_GRAPH_H: case KGE_TAP_GRAPH_R: case KGE_TAP_GRAPH_T: return h->graph_loaded ? (size_t)h->num_triples * 4 : 0;
        case KGE_TAP_GRAPH_OFF: case KGE_TAP_GRAPH_WCUM:
            return h->graph_loaded ? (size_t)c.num_parts * c.num_parts * (c.num_relations + 1) * 8 : 0;
        default: return 0;
    }
}

int kge_debug_export(kge_handle* h, int tap, void* dst, size_t bytes, void* stream) {
    if (!h || !dst) return KGE_ERR_BAD_ARG;
    if (!h->bound) return KGE_ERR_NOT_READY;
    const size_t want = kge_debug_bytes(h, tap, stream);
    if (want == 0 || want != bytes) return KGE_ERR_BAD_ARG;
    const Workspace& w = h->ws;
    const void* src = nullptr;
    switch (tap) {
        case KGE_TAP_Q: src = w.Q; break;
        case KGE_TAP_FPOS: src = w.fpos; break;
        case KGE_TAP_LROW: src = w.Lrow; break;
        case KGE_TAP_G: src = w.F; break;
        case KGE_TAP_GRAD_ENT: src = w.grad_ent; break;
        case KGE_TAP_GRAD_REL: src = w.grad_rel; break;
        case KGE_TAP_GRAD_RELW: src = w.grad_relw; break;
        case KGE_TAP_ENT_UNIQ: src = w.ent_uniq; break;
        case KGE_TAP_ENT_SEG: src = w.ent_seg; break;
        case KGE_TAP_ENT_PERM: src = w.ent_perm; break;
        case KGE_TAP_REL_UNIQ: src = w.rel_uniq; break;
        case KGE_TAP_REL_SEG: src = w.rel_seg; break;
        case KGE_TAP_REL_PERM: src = w.rel_perm; break;
        case KGE_TAP_BATCH: src = w.heads; break;
        case KGE_TAP_GRAPH_H: src = w.gh; break;
        case KGE_TAP_GRAPH_R: src = w.gr; break;
        case KGE_TAP_GRAPH_T: src = w.gt; break;
        case KGE_TAP_GRAPH_OFF: src = w.off; break;
        case KGE_TAP_GRAPH_WCUM: src = w.wcum; break;
        default: return KGE_ERR_BAD_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (tap == KGE_TAP_G && h->cfg.prec == KGE_PREC_BF16_TC) {
        // the tensor-core path keeps dL/dF only as bf16 [B, ldN]: widen it on the host
        const size_t B = h->cfg.batch, N = h->cfg.num_neg, ldN = (N + 7) / 8 * 8;
        std::vector<uint16_t> tmp(B * ldN);
        KGE_CUDA_CHECK(h, cudaMemcpyAsync(tmp.data(), w.Gb, tmp.size() * 2, cudaMemcpyDeviceToHost, s));
        KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
        float* out = static_cast<float*>(dst);
        for (size_t b = 0; b < B; ++b)
            for (size_t n = 0; n < N; ++n) {
                const uint32_t bits = (uint32_t)tmp[b * ldN + n] << 16;
                std::memcpy(&out[b * N + n], &bits, 4);
            }
        return KGE_OK;
    }
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    return KGE_OK;
}

}  // extern "C"
