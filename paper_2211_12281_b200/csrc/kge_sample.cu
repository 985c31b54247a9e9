// Balanced batch sampler (Section 4 "Training": Eq. 3, the cube-root relation law, Eq. 4):
// the stand-alone kernel behind kge_sample_batch.  One thread per slot.
#include "kge_sample.cuh"

namespace kge {

namespace {

constexpr int SAMPLE_THREADS = 128;

// CTAs [0, pos_ctas): positives.  A CTA serves SAMPLE_THREADS consecutive slots of ONE triple
// bucket, so the bucket's cumulative weights are fetched once, side by side, instead of by a
// chain of dependent reads per slot.  CTAs [pos_ctas, ...): negatives, one thread per slot.
__global__ void __launch_bounds__(SAMPLE_THREADS) sample_kernel(SampleParams p, int pos_ctas, int ctas_per_bucket,
                                                                int slots_per_bucket) {
    __shared__ uint64_t wsm[SAMPLE_SMEM_WEIGHTS];
    if ((int)blockIdx.x < pos_ctas) {
        const int bucket_slot = blockIdx.x / ctas_per_bucket;            // position of the bucket in the batch
        const int within = (blockIdx.x % ctas_per_bucket) * SAMPLE_THREADS + threadIdx.x;
        const int64_t base = sample_bucket_base(p, bucket_slot);
        const bool staged = p.sample_mode == 0 && p.R + 1 <= SAMPLE_SMEM_WEIGHTS;
        if (staged) {
            for (int r = threadIdx.x; r <= p.R; r += SAMPLE_THREADS) wsm[r] = p.wcum[base + r];
            __syncthreads();
        }
        if (within >= slots_per_bucket) return;
        const int slot = bucket_slot * slots_per_bucket + within;
        int32_t hh, rr, tt;
        sample_positive(p, slot, base, staged ? wsm : p.wcum + base, hh, rr, tt);
        p.heads[slot] = hh; p.rels[slot] = rr; p.tails[slot] = tt;
    } else {
        const int n = (blockIdx.x - pos_ctas) * SAMPLE_THREADS + threadIdx.x;
        if (n < p.N) p.negs[n] = sample_negative(p, n);
    }
}

}  // namespace

SampleParams make_sample_params(const kge_handle* h, uint64_t step) {
    const kge_config& c = h->cfg;
    SampleParams p;
    p.E = c.num_entities; p.R = c.num_relations; p.P = c.num_parts;
    p.S = (p.E + p.P - 1) / p.P;
    p.B = c.batch; p.N = c.num_neg; p.head_part = c.head_part; p.sample_mode = c.sample_mode;
    p.seed = c.seed; p.step = step;
    p.gh = h->ws.gh; p.gr = h->ws.gr; p.gt = h->ws.gt; p.off = h->ws.off; p.wcum = h->ws.wcum;
    p.heads = p.rels = p.tails = p.negs = nullptr;
    p.status = h->ws.status;
    return p;
}

int launch_sample(kge_handle* h, uint64_t step, int32_t* heads, int32_t* rels, int32_t* tails, int32_t* negs,
                  cudaStream_t s) {
    SampleParams p = make_sample_params(h, step);
    p.heads = heads; p.rels = rels; p.tails = tails; p.negs = negs;
    const int buckets = p.head_part < 0 ? p.P * p.P : p.P;     // buckets the batch draws from, in slot order
    const int slots_per_bucket = p.B / buckets;
    const int ctas_per_bucket = (slots_per_bucket + SAMPLE_THREADS - 1) / SAMPLE_THREADS;
    const int pos_ctas = buckets * ctas_per_bucket;
    const int neg_ctas = (p.N + SAMPLE_THREADS - 1) / SAMPLE_THREADS;
    stage_begin(h, ST_SAMPLE, s);
    sample_kernel<<<pos_ctas + neg_ctas, SAMPLE_THREADS, 0, s>>>(p, pos_ctas, ctas_per_bucket, slots_per_bucket);
    stage_end(h, ST_SAMPLE, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
