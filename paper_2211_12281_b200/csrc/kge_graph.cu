// Graph preprocessing on the device (Section 4 "Partitioning") and table initialisation.
//
// Graph: the triples are put in the canonical order "stable sort by (part(h), part(t), r)" with
// per-bucket relation offsets and running sums of the integer cube-root weights, exactly as the
// host path of kge_graph_load does, for triple lists that already live in device memory (600 M
// triples take minutes and three host copies on the host path).
//   key       : key(e) = (part(h) P + part(t)) R + r per triple, ids validated, keys counted
//               (integer atomics: the counts do not depend on the order)
//   scan      : exclusive scan of the counts -> first sorted index of every key
//   weights   : per bucket the offsets off[], the weights w_r = floor((n_r 2^60)^(1/3)) in 128-bit
//               integer arithmetic, and their running sums wcum[]
//   radix     : least-significant-digit radix sort of the triple INDICES by key, 8 bits per pass;
//               every pass is a stable split (tile histograms, one scan, ranks by warp votes in
//               input order), so equal keys keep the caller's order
//   gather    : h, r, t copied out in sorted order
// The three output arrays double as scratch: keys in gh, index buffers in gr and gt, the last
// pass lands in gt, which the gather overwrites in place last.
//
// Tables: Philox4x32-10 keyed by the seed with counter (row lo, row hi, c, stream) gives four
// words per group of four consecutive elements of a row; normal entries by Box-Muller on 23-bit
// uniforms (k + 1/2) 2^-23 (exactly representable in fp32), RotatE phases uniform in (-pi, pi).  A table is a pure function of (seed, stream).
#include <algorithm>
#include <cmath>

#include "kge_sample.cuh"

namespace kge {

namespace {

constexpr int RADIX_BITS = 8, RADIX = 1 << RADIX_BITS;
constexpr int RS_WARPS = 16, RS_THREADS = 32 * RS_WARPS;
constexpr int RS_ITEMS = 16;                                  // elements per lane and tile
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;                // 8192 elements per thread block

struct GraphParams {
    int64_t T, E, R, S, nkeys;
    int32_t P, head_part, sample_mode;
    const int32_t *h, *r, *t;          // caller's triples (device)
    int32_t *gh, *gr, *gt;             // outputs, also scratch
    unsigned long long* start;         // [nkeys + 1] counts, then first sorted index per key
    int64_t* off; uint64_t* wcum;      // [P * P * (R + 1)]
    uint32_t* hist;                    // [RADIX * tiles] digit-major tile histograms, then global offsets
    int32_t* flags;                    // [0] an id was out of range, [1] a bucket the sampler needs is empty
    int tiles;
};

__global__ void __launch_bounds__(256) graph_key_kernel(GraphParams p) {
    uint32_t* keys = reinterpret_cast<uint32_t*>(p.gh);
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < p.T; e += (int64_t)gridDim.x * blockDim.x) {
        const int32_t h = p.h[e], r = p.r[e], t = p.t[e];
        uint32_t key = 0;
        if (h < 0 || h >= p.E || t < 0 || t >= p.E || r < 0 || r >= p.R) {
            p.flags[0] = 1;
        } else {
            key = (uint32_t)(((int64_t)(h / p.S) * p.P + t / p.S) * p.R + r);
            atomicAdd(&p.start[key], 1ull);
        }
        keys[e] = key;
    }
}

// Exclusive scan of n counters in place by one thread block (each thread a contiguous share).
template <typename T>
__global__ void __launch_bounds__(1024) scan_kernel(T* a, int64_t n, int write_total) {
    __shared__ T warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t per = (n + 1023) / 1024;
    const int64_t i0 = min(n, (int64_t)tid * per), i1 = min(n, i0 + per);
    T sum = 0;
    for (int64_t i = i0; i < i1; ++i) sum += a[i];
    T incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    T before = 0, total = 0;
    for (int w = 0; w < 32; ++w) { if (w < warp) before += warp_tot[w]; total += warp_tot[w]; }
    T run = before + incl - sum;
    for (int64_t i = i0; i < i1; ++i) { const T v = a[i]; a[i] = run; run += v; }
    if (write_total && tid == 0) a[n] = total;
}

// Largest w with w^3 <= n * 2^60 (0 for n = 0): the integer cube-root sampling weight.
__device__ uint64_t icbrt_weight_dev(uint64_t n) {
    if (n == 0) return 0;
    const unsigned __int128 target = (unsigned __int128)n << 60;
    uint64_t lo = 0, hi = (uint64_t)1 << 42;
    while (lo < hi) {
        const uint64_t mid = lo + (hi - lo + 1) / 2;
        if ((unsigned __int128)mid * mid * mid <= target) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// One warp per bucket: offsets, weights, running sums in relation order.
__global__ void __launch_bounds__(256) graph_weights_kernel(GraphParams p) {
    const int b = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (b >= p.P * p.P) return;
    const unsigned long long* st = p.start + (int64_t)b * p.R;
    int64_t* off = p.off + (int64_t)b * (p.R + 1);
    uint64_t* wc = p.wcum + (int64_t)b * (p.R + 1);
    uint64_t carry = 0;
    for (int64_t r0 = 0; r0 < p.R; r0 += 32) {
        const int64_t r = r0 + lane;
        uint64_t w = 0;
        if (r < p.R) { off[r] = (int64_t)st[r]; w = icbrt_weight_dev(st[r + 1] - st[r]); }
        uint64_t incl = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint64_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (r < p.R) wc[r] = carry + incl - w;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
        off[p.R] = (int64_t)st[p.R];
        wc[p.R] = carry;
        const bool needed = p.head_part < 0 || b / p.P == p.head_part;
        const bool empty = p.sample_mode == 0 ? carry == 0 : st[p.R] == st[0];
        if (needed && empty) p.flags[1] = 1;
    }
}

// Digit of element i of this pass: the key of the triple that currently stands at position i.
__device__ __forceinline__ uint32_t radix_digit(const uint32_t* keys, const uint32_t* src, int64_t i, int shift, uint32_t& idx) {
    idx = src ? src[i] : (uint32_t)i;
    return (keys[idx] >> shift) & (RADIX - 1);
}

__global__ void __launch_bounds__(RS_THREADS) radix_hist_kernel(GraphParams p, const uint32_t* src, int shift) {
    __shared__ uint32_t hs[RADIX];
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(p.gh);
    for (int d = threadIdx.x; d < RADIX; d += RS_THREADS) hs[d] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * RS_TILE;
    for (int k = 0; k < RS_ITEMS; ++k) {
        const int64_t i = base + k * RS_THREADS + threadIdx.x;
        if (i < p.T) { uint32_t idx; atomicAdd(&hs[radix_digit(keys, src, i, shift, idx)], 1u); }
    }
    __syncthreads();
    for (int d = threadIdx.x; d < RADIX; d += RS_THREADS) p.hist[(int64_t)d * p.tiles + blockIdx.x] = hs[d];
}

// Stable split of one tile.  Warp w owns the tile's elements [w * 32 * RS_ITEMS, (w + 1) * 32 * RS_ITEMS)
// and takes them 32 at a time in order; within a round a lane's rank among the lanes with the same
// digit comes from a vote, across rounds from a running count per (warp, digit).  The counts of
// the warps are then turned into global positions (the scanned histogram gives where this tile's
// share of every digit starts), and every element is written to its place.
__global__ void __launch_bounds__(RS_THREADS) radix_scatter_kernel(GraphParams p, const uint32_t* src, uint32_t* dst, int shift) {
    __shared__ uint32_t cnt[RS_WARPS][RADIX];
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(p.gh);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int d = lane; d < RADIX; d += 32) cnt[warp][d] = 0;
    __syncwarp();
    const int64_t base = (int64_t)blockIdx.x * RS_TILE + (int64_t)warp * 32 * RS_ITEMS;
    uint32_t idx[RS_ITEMS], dr[RS_ITEMS];      // dr = digit << 16 | rank inside the warp's share (< 512)
#pragma unroll
    for (int k = 0; k < RS_ITEMS; ++k) {
        const int64_t i = base + k * 32 + lane;
        const bool in = i < p.T;
        uint32_t digit = RADIX;               // lanes beyond the list vote with a digit of their own
        idx[k] = 0;
        if (in) digit = radix_digit(keys, src, i, shift, idx[k]);
        const unsigned same = __match_any_sync(0xffffffffu, digit);
        const unsigned before = same & ((1u << lane) - 1u);
        uint32_t seen = 0;
        if (in) seen = cnt[warp][digit];
        __syncwarp();
        if (in && before == 0) cnt[warp][digit] = seen + __popc(same);     // the first lane of the group keeps the count
        __syncwarp();
        dr[k] = (digit << 16) | (seen + __popc(before));
    }
    __syncthreads();
    for (int d = threadIdx.x; d < RADIX; d += RS_THREADS) {
        uint32_t run = p.hist[(int64_t)d * p.tiles + blockIdx.x];
        for (int w = 0; w < RS_WARPS; ++w) { const uint32_t c = cnt[w][d]; cnt[w][d] = run; run += c; }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < RS_ITEMS; ++k) {
        const int64_t i = base + k * 32 + lane;
        if (i < p.T) dst[cnt[warp][dr[k] >> 16] + (dr[k] & 0xffffu)] = idx[k];
    }
}

__global__ void __launch_bounds__(256) graph_gather_kernel(GraphParams p) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < p.T; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t j = reinterpret_cast<const uint32_t*>(p.gt)[i];
        p.gh[i] = p.h[j]; p.gr[i] = p.r[j]; p.gt[i] = p.t[j];
    }
}

// ---- table initialisation ----
struct InitParams { float* out; int64_t rows; int width; float std; int kind; uint32_t stream; uint64_t seed; };

__global__ void __launch_bounds__(256) init_table_kernel(InitParams p) {
    const int groups = (p.width + 3) / 4;
    const int64_t total = p.rows * groups;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = g / groups;
        const int c = (int)(g - row * groups);
        const Philox4 o = philox4x32_10((uint32_t)row, (uint32_t)((uint64_t)row >> 32), (uint32_t)c, p.stream,
                                        (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
        const uint32_t x[4] = {o.x, o.y, o.z, o.w};
        float v[4];
        if (p.kind == 2) {                       // the raw words, as bit patterns (parity tap of the generator)
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = __uint_as_float(x[j]);
        } else {
            float u[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) u[j] = ((float)(x[j] >> 9) + 0.5f) * 1.1920928955078125e-07f;   // (k + 1/2) 2^-23, exact in fp32: u in (0, 1)
            if (p.kind == 1) {
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = (2.f * u[j] - 1.f) * 3.14159265358979323846f;
            } else {
#pragma unroll
                for (int j = 0; j < 4; j += 2) {
                    const float rad = p.std * sqrtf(-2.f * logf(u[j]));
                    float sn, cs;
                    sincosf(6.28318530717958647692f * u[j + 1], &sn, &cs);
                    v[j] = rad * cs; v[j + 1] = rad * sn;
                }
            }
        }
        float* dst = p.out + row * p.width + 4 * c;
#pragma unroll
        for (int j = 0; j < 4; ++j) if (4 * c + j < p.width) dst[j] = v[j];
    }
}

int grid_for(int64_t n, int threads, int num_sms) {
    return (int)std::max<int64_t>(1, std::min<int64_t>((n + threads - 1) / threads, (int64_t)num_sms * 32));
}

}  // namespace

int graph_radix_tiles(int64_t num_triples) { return (int)((num_triples + RS_TILE - 1) / RS_TILE); }
size_t graph_hist_words(int64_t num_triples) { return (size_t)RADIX * graph_radix_tiles(num_triples) + 1; }

int launch_graph_build_device(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails, int64_t n,
                              cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    GraphParams p;
    p.T = n; p.E = c.num_entities; p.R = c.num_relations; p.P = c.num_parts;
    p.S = (p.E + p.P - 1) / p.P;
    p.nkeys = (int64_t)p.P * p.P * p.R;
    p.head_part = c.head_part; p.sample_mode = c.sample_mode;
    p.h = heads; p.r = rels; p.t = tails;
    p.gh = w.gh; p.gr = w.gr; p.gt = w.gt;
    p.start = reinterpret_cast<unsigned long long*>(w.gstart);
    p.off = w.off; p.wcum = w.wcum; p.hist = w.ghist;
    p.flags = w.status + 2;
    p.tiles = graph_radix_tiles(n);
    KGE_CUDA_CHECK(h, cudaMemsetAsync(p.start, 0, (size_t)(p.nkeys + 1) * sizeof(unsigned long long), s));
    KGE_CUDA_CHECK(h, cudaMemsetAsync(p.flags, 0, 2 * sizeof(int32_t), s));
    graph_key_kernel<<<grid_for(n, 256, h->num_sms), 256, 0, s>>>(p);
    KGE_LAUNCH_CHECK(h);
    scan_kernel<unsigned long long><<<1, 1024, 0, s>>>(p.start, p.nkeys, 1);
    KGE_LAUNCH_CHECK(h);
    graph_weights_kernel<<<(p.P * p.P * 32 + 255) / 256, 256, 0, s>>>(p);
    KGE_LAUNCH_CHECK(h);
    int bits = 0;
    while (((int64_t)1 << bits) < p.nkeys) ++bits;
    const int passes = std::max(1, (bits + RADIX_BITS - 1) / RADIX_BITS);
    const uint32_t* src = nullptr;             // pass 0 reads the identity order
    for (int pass = 0; pass < passes; ++pass) {
        // the index buffers alternate so that the last pass writes gt
        uint32_t* dst = reinterpret_cast<uint32_t*>(((passes - 1 - pass) % 2 == 0) ? w.gt : w.gr);
        if (n > 0) {
            radix_hist_kernel<<<p.tiles, RS_THREADS, 0, s>>>(p, src, pass * RADIX_BITS);
            KGE_LAUNCH_CHECK(h);
            scan_kernel<uint32_t><<<1, 1024, 0, s>>>(p.hist, (int64_t)RADIX * p.tiles, 0);
            KGE_LAUNCH_CHECK(h);
            radix_scatter_kernel<<<p.tiles, RS_THREADS, 0, s>>>(p, src, dst, pass * RADIX_BITS);
            KGE_LAUNCH_CHECK(h);
        }
        src = dst;
    }
    if (n > 0) {
        graph_gather_kernel<<<grid_for(n, 256, h->num_sms), 256, 0, s>>>(p);
        KGE_LAUNCH_CHECK(h);
    }
    int32_t flags[2] = {0, 0};
    KGE_CUDA_CHECK(h, cudaMemcpyAsync(flags, p.flags, sizeof(flags), cudaMemcpyDeviceToHost, s));
    KGE_CUDA_CHECK(h, cudaStreamSynchronize(s));
    if (flags[0]) return KGE_ERR_BAD_ARG;
    if (flags[1]) return KGE_ERR_EMPTY_BUCKET;
    return KGE_OK;
}

int launch_init_table(kge_handle* h, float* out, int64_t rows, int width, float std, int kind, uint32_t stream_id, cudaStream_t s) {
    InitParams p{out, rows, width, std, kind, stream_id, h->cfg.seed};
    const int64_t groups = rows * ((width + 3) / 4);
    init_table_kernel<<<grid_for(groups, 256, h->num_sms), 256, 0, s>>>(p);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
