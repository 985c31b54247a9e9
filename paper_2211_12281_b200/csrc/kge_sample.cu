// Balanced batch sampler (Section 4 "Training": Eq. 3, the cube-root relation law, Eq. 4).
// One thread per slot; random words from Philox4x32-10 keyed by the seed with counter
// (slot, step lo, step hi, stream), so a batch is a pure function of (seed, step).
#include "kge_common.cuh"

namespace kge {

namespace {

struct Philox4 { uint32_t x, y, z, w; };

// Philox4x32 with 10 rounds (Salmon et al., SC'11).
__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return Philox4{c0, c1, c2, c3};
}

struct SampleParams {
    int64_t E, R, S;
    int32_t P, B, N, head_part, sample_mode;
    uint64_t seed, step;
    const int32_t *gh, *gr, *gt;
    const int64_t* off;
    const uint64_t* wcum;
    int32_t *heads, *rels, *tails, *negs;
    int32_t* status;
};

constexpr int SAMPLE_THREADS = 128;
constexpr int SAMPLE_SMEM_WEIGHTS = 4096;   // cumulative weights of up to 4095 relations are staged in shared memory

// CTAs [0, pos_ctas): positives.  A CTA serves SAMPLE_THREADS consecutive slots of ONE triple
// bucket, so the bucket's cumulative weights are fetched once, side by side, instead of by a
// chain of dependent reads per slot.  CTAs [pos_ctas, ...): negatives, one thread per slot.
__global__ void __launch_bounds__(SAMPLE_THREADS) sample_kernel(SampleParams p, int pos_ctas, int ctas_per_bucket,
                                                                int slots_per_bucket) {
    __shared__ uint64_t wsm[SAMPLE_SMEM_WEIGHTS];
    const uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
    const uint32_t s0 = (uint32_t)p.step, s1 = (uint32_t)(p.step >> 32);
    if ((int)blockIdx.x < pos_ctas) {
        const int bucket_slot = blockIdx.x / ctas_per_bucket;            // position of the bucket in the batch
        const int within = (blockIdx.x % ctas_per_bucket) * SAMPLE_THREADS + threadIdx.x;
        const int i = p.head_part < 0 ? bucket_slot / p.P : p.head_part;
        const int j = p.head_part < 0 ? bucket_slot % p.P : bucket_slot;
        const int64_t base = ((int64_t)i * p.P + j) * (p.R + 1);
        const bool staged = p.sample_mode == 0 && p.R + 1 <= SAMPLE_SMEM_WEIGHTS;
        if (staged) {
            for (int r = threadIdx.x; r <= p.R; r += SAMPLE_THREADS) wsm[r] = p.wcum[base + r];
            __syncthreads();
        }
        if (within >= slots_per_bucket) return;
        const int slot = bucket_slot * slots_per_bucket + within;
        const Philox4 o = philox4x32_10((uint32_t)slot, s0, s1, 0u, k0, k1);
        const uint64_t x64 = (uint64_t)o.x | ((uint64_t)o.y << 32);
        const uint64_t y64 = (uint64_t)o.z | ((uint64_t)o.w << 32);
        int64_t idx;
        if (p.sample_mode == 0) {
            const uint64_t* wc = staged ? wsm : p.wcum + base;
            const uint64_t u = __umul64hi(x64, wc[p.R]);
            // largest r with wcum[r] <= u; relations with weight 0 own an empty interval
            int64_t lo = 0, hi = p.R - 1;
            while (lo < hi) {
                const int64_t mid = (lo + hi + 1) >> 1;
                if (wc[mid] <= u) lo = mid; else hi = mid - 1;
            }
            const int64_t first = p.off[base + lo];
            const uint64_t n_r = (uint64_t)(p.off[base + lo + 1] - first);
            idx = first + (int64_t)__umul64hi(y64, n_r);
        } else {
            const int64_t first = p.off[base];
            idx = first + (int64_t)__umul64hi(x64, (uint64_t)(p.off[base + p.R] - first));
        }
        p.heads[slot] = p.gh[idx]; p.rels[slot] = p.gr[idx]; p.tails[slot] = p.gt[idx];
    } else {
        const int n = (blockIdx.x - pos_ctas) * SAMPLE_THREADS + threadIdx.x;
        if (n >= p.N) return;
        const int j = n / (p.N / p.P);
        int64_t size_j = p.E - (int64_t)j * p.S;
        if (size_j > p.S) size_j = p.S;
        const Philox4 o = philox4x32_10((uint32_t)n, s0, s1, 1u, k0, k1);
        const uint64_t x64 = (uint64_t)o.x | ((uint64_t)o.y << 32);
        p.negs[n] = (int32_t)((int64_t)j * p.S + (int64_t)__umul64hi(x64, (uint64_t)size_j));
    }
}

}  // namespace

int launch_sample(kge_handle* h, uint64_t step, int32_t* heads, int32_t* rels, int32_t* tails, int32_t* negs,
                  cudaStream_t s) {
    const kge_config& c = h->cfg;
    SampleParams p;
    p.E = c.num_entities; p.R = c.num_relations; p.P = c.num_parts;
    p.S = (p.E + p.P - 1) / p.P;
    p.B = c.batch; p.N = c.num_neg; p.head_part = c.head_part; p.sample_mode = c.sample_mode;
    p.seed = c.seed; p.step = step;
    p.gh = h->ws.gh; p.gr = h->ws.gr; p.gt = h->ws.gt; p.off = h->ws.off; p.wcum = h->ws.wcum;
    p.heads = heads; p.rels = rels; p.tails = tails; p.negs = negs;
    p.status = h->ws.status;
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
