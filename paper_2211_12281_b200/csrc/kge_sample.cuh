// Device side of the balanced batch sampler (Section 4 "Training": Eq. 3, the cube-root relation
// law, Eq. 4), shared by the stand-alone sampling kernel and the gather kernel that draws its own
// batch.  Random words come from Philox4x32-10 keyed by the seed with counter (slot, step lo,
// step hi, stream): a batch is a pure function of (seed, step).
#pragma once

#include "kge_common.cuh"

namespace kge {

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


// Bucket (i, j) that batch slot `bucket_slot`-th group of slots draws from.
__device__ __forceinline__ int64_t sample_bucket_base(const SampleParams& p, int bucket_slot) {
    const int i = p.head_part < 0 ? bucket_slot / p.P : p.head_part;
    const int j = p.head_part < 0 ? bucket_slot % p.P : bucket_slot;
    return ((int64_t)i * p.P + j) * (p.R + 1);
}

// Positive of batch slot `slot`, drawn from the bucket whose rows of `off` / `wcum` start at
// `base`; `wc` = that bucket's cumulative weights (shared or global memory).
__device__ __forceinline__ void sample_positive(const SampleParams& p, int slot, int64_t base, const uint64_t* wc,
                                                int32_t& h, int32_t& r, int32_t& t) {
    const Philox4 o = philox4x32_10((uint32_t)slot, (uint32_t)p.step, (uint32_t)(p.step >> 32), 0u,
                                    (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
    const uint64_t x64 = (uint64_t)o.x | ((uint64_t)o.y << 32);
    const uint64_t y64 = (uint64_t)o.z | ((uint64_t)o.w << 32);
    int64_t idx;
    if (p.sample_mode == 0) {
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
    h = p.gh[idx]; r = p.gr[idx]; t = p.gt[idx];
}

// Negative of slot n: uniform in partition n div (N / P).
__device__ __forceinline__ int32_t sample_negative(const SampleParams& p, int n) {
    const int j = n / (p.N / p.P);
    int64_t size_j = p.E - (int64_t)j * p.S;
    if (size_j > p.S) size_j = p.S;
    const Philox4 o = philox4x32_10((uint32_t)n, (uint32_t)p.step, (uint32_t)(p.step >> 32), 1u,
                                    (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
    const uint64_t x64 = (uint64_t)o.x | ((uint64_t)o.y << 32);
    return (int32_t)((int64_t)j * p.S + (int64_t)__umul64hi(x64, (uint64_t)size_j));
}

constexpr int SAMPLE_SMEM_WEIGHTS = 4096;   // cumulative weights of up to 4095 relations are staged in shared memory

// Fills the sampler's parameters from the handle (outputs left to the caller).
SampleParams make_sample_params(const kge_handle* h, uint64_t step);

}  // namespace kge
