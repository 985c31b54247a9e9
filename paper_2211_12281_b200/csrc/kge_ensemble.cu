// Power-rank ensemble (Section 3.2 "Ensemble", Eq. 2): M models each give a top-K list of tails per
// query; an entity's ensemble score is the sum over the models of a rank-based score,
//     s_m(t) = -sgn(p) k^p            if t is the k-th entry of model m's list (k = 1 .. K)
//              -[p > 0] (K + 1)^p     if t is not in model m's list,
// and the query's final prediction is the top-n entities by s(t) (ties: smaller entity id first).
// Only entities that occur in some list can reach the top (an entity in no list has the lowest
// possible score and every list holds K >= n distinct entities), so the candidates of a query are
// the union of its M lists.
//
// One thread block per query.  The M * K list entries are sorted in shared memory by (entity id,
// model, position); the first entry of every run of equal ids adds the run's rank scores model by
// model in ascending model order (an absent model contributes the absent score at its place in that
// order), in fp64; n rounds of a block-wide maximum then pick the result.  The rank scores k^p come
// from a table the caller fills with kge_ensemble_rank_scores, so the sums are plain IEEE additions
// of given numbers in a fixed order: the result does not depend on any device math library.
#include <cmath>

#include "kge_common.cuh"

namespace kge {
namespace {

constexpr int ENS_THREADS = 512;
constexpr int ENS_MAX_ENTRIES = 16384;      // M * K per query (85 models x top-100 = 8,500 fits)

struct EnsParams {
    const int32_t* lists;      // [M, nq, K]
    const double* table;       // [K + 1]: rank scores of positions 1 .. K, then the absent score
    int M, nq, K, top_n, n2;   // n2 = M * K rounded up to a power of two
    int32_t* out_ids; double* out_scores;
};

__device__ __forceinline__ bool ens_before(double sa, int32_t ia, double sb, int32_t ib) { return sa > sb || (sa == sb && ia < ib); }

__global__ void __launch_bounds__(ENS_THREADS) ensemble_kernel(EnsParams p) {
    extern __shared__ __align__(16) unsigned char ens_smem[];
    uint64_t* key = reinterpret_cast<uint64_t*>(ens_smem);                      // [n2] (id, model, position); later the candidates' scores
    int32_t* cid = reinterpret_cast<int32_t*>(key + p.n2);                      // [n2] candidate id at the first entry of its run, else -1
    __shared__ double red_s[ENS_THREADS / 32];
    __shared__ int32_t red_i[ENS_THREADS / 32], red_pos[ENS_THREADS / 32];
    __shared__ int32_t win_pos;
    const int q = blockIdx.x, tid = threadIdx.x, n = p.M * p.K;
    for (int i = tid; i < p.n2; i += ENS_THREADS) {
        uint64_t k = ~0ull;
        if (i < n) {
            const int m = i / p.K, pos = i - m * p.K;
            const int32_t id = p.lists[((int64_t)m * p.nq + q) * p.K + pos];
            if (id >= 0) k = ((uint64_t)(uint32_t)id << 32) | ((uint64_t)m << 16) | (uint64_t)pos;   // unused places of a list hold -1
        }
        key[i] = k;
    }
    __syncthreads();
    for (int size = 2; size <= p.n2; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = tid; t < p.n2 / 2; t += ENS_THREADS) {
                const int lo = 2 * t - (t & (stride - 1)), hi = lo + stride;
                const bool up = (lo & size) == 0;
                const uint64_t x = key[lo], y = key[hi];
                if ((x > y) == up) { key[lo] = y; key[hi] = x; }
            }
            __syncthreads();
        }
    // runs of equal ids: mark their first entries (reads only)
    for (int i = tid; i < p.n2; i += ENS_THREADS) {
        const uint64_t k = key[i];
        const bool head = k != ~0ull && (i == 0 || (key[i - 1] >> 32) != (k >> 32));
        cid[i] = head ? (int32_t)(k >> 32) : -1;
    }
    __syncthreads();
    // every run is summed by the thread of its first entry, which then keeps the score in that entry's place
    const double absent = p.table[p.K];
    for (int i = tid; i < p.n2; i += ENS_THREADS) {
        if (cid[i] < 0) continue;
        const uint32_t id = (uint32_t)cid[i];
        int j = i;
        double s = 0.0;
        for (int m = 0; m < p.M; ++m) {
            bool present = false;
            while (j < p.n2 && (uint32_t)(key[j] >> 32) == id && (int)((key[j] >> 16) & 0xffffu) == m) {
                s += p.table[key[j] & 0xffffu];
                present = true; ++j;
            }
            if (!present) s += absent;
        }
        key[i] = (uint64_t)__double_as_longlong(s);
    }
    __syncthreads();
    for (int r = 0; r < p.top_n; ++r) {
        double bs = -INFINITY; int32_t bi = INT32_MAX, bp = -1;
        for (int i = tid; i < p.n2; i += ENS_THREADS) {
            const int32_t id = cid[i];
            if (id < 0) continue;
            const double s = __longlong_as_double((long long)key[i]);
            if (bp < 0 || ens_before(s, id, bs, bi)) { bs = s; bi = id; bp = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double os = __shfl_xor_sync(0xffffffffu, bs, o);
            const int32_t oi = __shfl_xor_sync(0xffffffffu, bi, o), op = __shfl_xor_sync(0xffffffffu, bp, o);
            if (op >= 0 && (bp < 0 || ens_before(os, oi, bs, bi))) { bs = os; bi = oi; bp = op; }
        }
        if ((tid & 31) == 0) { red_s[tid >> 5] = bs; red_i[tid >> 5] = bi; red_pos[tid >> 5] = bp; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < ENS_THREADS / 32; ++w)
                if (red_pos[w] >= 0 && (bp < 0 || ens_before(red_s[w], red_i[w], bs, bi))) { bs = red_s[w]; bi = red_i[w]; bp = red_pos[w]; }
            p.out_ids[(int64_t)q * p.top_n + r] = bp >= 0 ? bi : -1;          // fewer candidates than places: -1 and -inf
            if (p.out_scores) p.out_scores[(int64_t)q * p.top_n + r] = bp >= 0 ? bs : -INFINITY;
            win_pos = bp;
        }
        __syncthreads();
        if (tid == 0 && win_pos >= 0) cid[win_pos] = -1;                       // taken
        __syncthreads();
    }
}

}  // namespace
}  // namespace kge

extern "C" {

int kge_ensemble_rank_scores(double power, int32_t k_list, double* table) {
    if (!table || k_list <= 0 || power == 0.0 || !std::isfinite(power)) return KGE_ERR_BAD_ARG;
    const double sign = power > 0.0 ? 1.0 : -1.0;
    for (int32_t k = 1; k <= k_list; ++k) table[k - 1] = -sign * std::pow((double)k, power);
    table[k_list] = power > 0.0 ? -std::pow((double)k_list + 1.0, power) : 0.0;
    return KGE_OK;
}

int kge_ensemble_topk(const int32_t* lists, int32_t num_models, int32_t nq, int32_t k_list, const double* table,
                      int32_t top_n, int32_t* out_ids, double* out_scores, void* stream) {
    using namespace kge;
    if (!lists || !table || !out_ids || num_models <= 0 || nq < 0 || k_list <= 0 || top_n <= 0) return KGE_ERR_BAD_ARG;
    if (num_models > 65535 || k_list > 65535) return KGE_ERR_UNSUPPORTED;
    if ((int64_t)num_models * k_list > ENS_MAX_ENTRIES) return KGE_ERR_WORKSPACE;
    if (nq == 0) return KGE_OK;
    EnsParams p;
    p.lists = lists; p.table = table; p.M = num_models; p.nq = nq; p.K = k_list; p.top_n = top_n;
    p.n2 = 2;
    while (p.n2 < num_models * k_list) p.n2 <<= 1;
    p.out_ids = out_ids; p.out_scores = out_scores;
    const size_t smem = (size_t)p.n2 * (sizeof(uint64_t) + sizeof(int32_t));
    static DeviceOnce configured;
    cudaError_t e = once_per_device(configured, [] {
        return cudaFuncSetAttribute(ensemble_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)(ENS_MAX_ENTRIES * (sizeof(uint64_t) + sizeof(int32_t))));
    });
    if (e != cudaSuccess) return KGE_ERR_CUDA;
    ensemble_kernel<<<nq, ENS_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? KGE_OK : KGE_ERR_CUDA;
}

}  // extern "C"
