// Deterministic de-duplication of touched rows and the sparse row update.
//   tile_sort : every 1024 ids of a list, tagged with their source position, sorted in shared memory
//   rank      : global stable rank of each id = sum over tiles of (keys below it); scatter to
//               the permutation and the sorted id list
//   segment   : distinct ids, segment offsets, segment index of every sorted position
//               (single-CTA scan), batch loss reduction
//   piece     : one warp per sorted position; a segment of at most 16 rows is summed in
//               ascending source position by the warp at its first position and the row is
//               updated at once (SGD / Adam / row-wise Adagrad); a longer segment is cut
//               into pieces of 16 rows, each summed by its own warp into a partial row, and
//               the warp that finishes the last outstanding piece adds the pieces in
//               ascending order and updates the row
// The summation order of a segment is therefore fixed by the batch alone: results are
// bit-reproducible, and a row that occurs hundreds of times in a batch does not serialise
// behind a single warp.
#include <cmath>

#include "kge_common.cuh"

namespace kge {

namespace {

constexpr int SORT_TILE = 1024;      // keys per shared-memory sort
constexpr int SORT_THREADS = 512;
constexpr int RANK_THREADS = 256;
constexpr int SEG_THREADS = 1024;
constexpr int PIECE = 16;            // gradient rows summed by one warp in one go

struct IdList {
    const int32_t *a, *b, *c;   // the list is the concatenation a[0..na) | b[0..nb) | c[0..nc)
    int na, nb, nc;
    int64_t rows;               // table rows (ids outside [0, rows) are reported and read as 0)
    int32_t *perm, *sorted, *uniq, *seg, *seg_of;
    int32_t *seg_done, *seg_done2;   // [n] pieces finished per long segment (zeroed here for the update kernel); second table on the same list, or NULL
    uint64_t* tkeys;            // [tiles * SORT_TILE] tile-sorted (id << 32 | position), padded with ~0
    int32_t* count;             // number of distinct ids
    __host__ __device__ __forceinline__ int n() const { return na + nb + nc; }
    __device__ __forceinline__ int32_t raw(int i) const {
        return i < na ? a[i] : (i < na + nb ? b[i - na] : c[i - na - nb]);
    }
};

struct DedupParams {
    IdList ent, rel;
    int ent_tiles;              // sort / rank kernels: tiles [0, ent_tiles) serve the entity list
    int32_t* status;
};

__global__ void __launch_bounds__(SORT_THREADS) tile_sort_kernel(DedupParams p) {
    __shared__ uint64_t k[SORT_TILE];
    const bool is_ent = (int)blockIdx.x < p.ent_tiles;
    const IdList& L = is_ent ? p.ent : p.rel;
    const int tile = is_ent ? blockIdx.x : blockIdx.x - p.ent_tiles;
    const int n = L.n(), tid = threadIdx.x;
    for (int j = tid; j < SORT_TILE; j += SORT_THREADS) {
        const int i = tile * SORT_TILE + j;
        uint64_t key = ~0ull;
        if (i < n) key = ((uint64_t)(uint32_t)checked_id(L.raw(i), L.rows, p.status) << 32) | (uint32_t)i;
        k[j] = key;
    }
    __syncthreads();
    for (int size = 2; size <= SORT_TILE; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const int lo = 2 * tid - (tid & (stride - 1)), hi = lo + stride;
            const bool up = (lo & size) == 0;
            const uint64_t x = k[lo], y = k[hi];
            if ((x > y) == up) { k[lo] = y; k[hi] = x; }
            __syncthreads();
        }
    }
    for (int j = tid; j < SORT_TILE; j += SORT_THREADS) L.tkeys[(int64_t)tile * SORT_TILE + j] = k[j];
}

// Keys are distinct (the position is part of the key), so "number of keys below mine" summed
// over all tiles is the position of the key in the stable sort by id.
__global__ void __launch_bounds__(RANK_THREADS) rank_kernel(DedupParams p) {
    __shared__ uint64_t sk[SORT_TILE];
    constexpr int PER_TILE = SORT_TILE / RANK_THREADS;
    int blk = blockIdx.x;
    const bool is_ent = blk < p.ent_tiles * PER_TILE;
    const IdList& L = is_ent ? p.ent : p.rel;
    if (!is_ent) blk -= p.ent_tiles * PER_TILE;
    const int tile = blk / PER_TILE, j = (blk % PER_TILE) * RANK_THREADS + threadIdx.x;
    const int n = L.n(), tiles = (n + SORT_TILE - 1) / SORT_TILE;
    const uint64_t key = L.tkeys[(int64_t)tile * SORT_TILE + j];
    int rank = j;
    for (int t = 0; t < tiles; ++t) {
        if (t == tile) continue;
        __syncthreads();
        for (int x = threadIdx.x; x < SORT_TILE; x += RANK_THREADS) sk[x] = L.tkeys[(int64_t)t * SORT_TILE + x];
        __syncthreads();
        int lo = 0;
#pragma unroll
        for (int step = SORT_TILE >> 1; step >= 1; step >>= 1) lo += (sk[lo + step - 1] < key) ? step : 0;
        lo += (sk[lo] < key) ? 1 : 0;
        rank += lo;
    }
    if (key != ~0ull) { L.perm[rank] = (int32_t)(uint32_t)key; L.sorted[rank] = (int32_t)(key >> 32); }
}

// blockIdx.x = 0: entity list, 1: relation list.  One CTA walks the sorted list 1024 positions at a
// time (coalesced reads): a position opens a segment if its id differs from the one before it, and
// the number of openings up to a position (a ballot scan inside each warp, warp totals through
// shared memory, a running carry between rounds) is the index of its segment.
__global__ void __launch_bounds__(SEG_THREADS) segment_kernel(DedupParams p) {
    __shared__ int32_t warp_tot[SEG_THREADS / 32];
    __shared__ int32_t carry_sm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const IdList& L = blockIdx.x == 0 ? p.ent : p.rel;
    const int n = L.n();
    if (tid == 0) carry_sm = 0;
    __syncthreads();
    // (ids are non-negative: position 0 opens a segment; the next round's ids are requested before this round's scan)
    auto id_at = [&](int r) { return (r >= 0 && r < n) ? L.sorted[r] : -1; };
    int32_t id_nx = id_at(tid), prev_nx = id_at(tid - 1);
    for (int base = 0; base < n; base += SEG_THREADS) {
        const int r = base + tid;
        const int32_t id = id_nx, prev = prev_nx;
        id_nx = id_at(r + SEG_THREADS); prev_nx = id_at(r + SEG_THREADS - 1);
        const bool head = r < n && id != prev;
        const unsigned mask = __ballot_sync(0xffffffffu, head);
        const int incl = __popc(mask & (0xffffffffu >> (31 - lane)));
        if (lane == 0) warp_tot[warp] = __popc(mask);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < SEG_THREADS / 32; ++w) { const int t = warp_tot[w]; if (w < warp) before += t; total += t; }
        const int carry = carry_sm;
        if (r < n) {
            const int u = carry + before + incl - 1;
            if (head) { L.uniq[u] = id; L.seg[u] = r; }
            L.seg_of[r] = u;
            L.seg_done[r] = 0;
            if (L.seg_done2) L.seg_done2[r] = 0;
        }
        __syncthreads();
        if (tid == 0) carry_sm = carry + total;
        __syncthreads();
    }
    if (tid == 0) { L.seg[carry_sm] = n; *L.count = carry_sm; }
}

struct UpdateJob {
    float* table; float* state;        // [rows, width], optimiser state
    const float* grads;                // [n, width] gradient rows by source position
    float* part;                       // [n, width] partial sums of long segments, row = first sorted position of the piece
    const int32_t *uniq, *seg, *perm, *sorted, *seg_of;
    int32_t* seg_done;                 // [n] per segment: pieces of a long segment that have been written
    int width, n;                      // n = list length
};

struct UpdateParams {
    UpdateJob job[3];
    int njobs;
    int warp_begin[4];                 // job j serves warps [warp_begin[j], warp_begin[j+1]): one per sorted position
    int opt;
    float lr, beta1, beta2, eps, corr1, corr2;   // corr = 1 - beta^t
};

__device__ __forceinline__ float approx_sqrt(float x) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float approx_rcp(float x) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

template <typename V> struct VecOps;
template <> struct VecOps<float> {
    static constexpr int LEN = 1;
    static __device__ __forceinline__ float zero() { return 0.f; }
    static __device__ __forceinline__ void add(float& a, float b) { a += b; }
};
template <> struct VecOps<float4> {
    static constexpr int LEN = 4;
    static __device__ __forceinline__ float4 zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
    static __device__ __forceinline__ void add(float4& a, float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
};

// One optimiser step on table row `row` with the summed gradient g (lane l holds elements
// l, l + 32, ... of the row in units of V).
template <typename V, int NCH>
__device__ __forceinline__ void apply_row(const UpdateJob& J, const UpdateParams& p, int64_t row, V (&g)[NCH], int lane) {
    constexpr int LEN = VecOps<V>::LEN;
    const int wv = J.width / LEN;
    V* prow = reinterpret_cast<V*>(J.table) + row * wv;
    if (p.opt == KGE_OPT_SGD) {
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = lane + 32 * i;
            if (c < wv) {
                V v = prow[c];
                float* vv = reinterpret_cast<float*>(&v); const float* gg = reinterpret_cast<const float*>(&g[i]);
#pragma unroll
                for (int e = 0; e < LEN; ++e) vv[e] -= p.lr * gg[e];
                prow[c] = v;
            }
        }
    } else if (p.opt == KGE_OPT_ADAM) {
        V* mrow = reinterpret_cast<V*>(J.state) + row * 2 * wv;
        V* vrow = mrow + wv;
        const float inv_corr1 = 1.f / p.corr1, inv_corr2 = 1.f / p.corr2;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = lane + 32 * i;
            if (c < wv) {
                V m = mrow[c], v = vrow[c], x = prow[c];
                float* mm = reinterpret_cast<float*>(&m); float* vv = reinterpret_cast<float*>(&v);
                float* xx = reinterpret_cast<float*>(&x); const float* gg = reinterpret_cast<const float*>(&g[i]);
#pragma unroll
                for (int e = 0; e < LEN; ++e) {
                    mm[e] = p.beta1 * mm[e] + (1.f - p.beta1) * gg[e];
                    vv[e] = p.beta2 * vv[e] + (1.f - p.beta2) * gg[e] * gg[e];
                    // one special-function instruction for the square root and one for the reciprocal (relative
                    // error about 2^-22 on the step): the correctly rounded forms are some forty dependent
                    // instructions per element and made this kernel wait on arithmetic, not on memory
                    xx[e] = fmaf(-(p.lr * inv_corr1) * mm[e], approx_rcp(approx_sqrt(vv[e] * inv_corr2) + p.eps), xx[e]);
                }
                mrow[c] = m; vrow[c] = v; prow[c] = x;
            }
        }
    } else {
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const float* gg = reinterpret_cast<const float*>(&g[i]);
#pragma unroll
            for (int e = 0; e < LEN; ++e) ss += gg[e] * gg[e];   // lanes beyond the row hold zeros
        }
        ss = warp_sum(ss) / (float)J.width;
        const float acc = J.state[row] + ss;
        __syncwarp();
        if (lane == 0) J.state[row] = acc;
        const float step = p.lr / (sqrtf(acc) + p.eps);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = lane + 32 * i;
            if (c < wv) {
                V v = prow[c];
                float* vv = reinterpret_cast<float*>(&v); const float* gg = reinterpret_cast<const float*>(&g[i]);
#pragma unroll
                for (int e = 0; e < LEN; ++e) vv[e] -= step * gg[e];
                prow[c] = v;
            }
        }
    }
}

// g += rows[idx[0]], rows[idx[1]], ... in that order, a few rows' loads in flight at a time
// (four for narrow rows, two for wide ones, to keep the register count down).
// FRESH: the rows were written by other warps of this launch; read them past the L1 cache.
template <typename V, int NCH, bool FRESH = false, typename IndexOf>
__device__ __forceinline__ void ordered_sum(const V* rows, int wv, int count, IndexOf index_of, V (&g)[NCH], int lane) {
    constexpr int BATCH = NCH == 1 ? 4 : 2;
    for (int s = 0; s < count; s += BATCH) {
        V v[BATCH][NCH];
#pragma unroll
        for (int r = 0; r < BATCH; ++r) {
            const V* src = rows + (s + r < count ? index_of(s + r) : 0) * wv;
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                const int c = lane + 32 * i;
                v[r][i] = (s + r < count && c < wv) ? (FRESH ? __ldcg(src + c) : src[c]) : VecOps<V>::zero();
            }
        }
#pragma unroll
        for (int r = 0; r < BATCH; ++r)
#pragma unroll
            for (int i = 0; i < NCH; ++i) VecOps<V>::add(g[i], v[r][i]);
    }
}

// One warp per sorted position.  A warp whose position opens a segment of at most PIECE rows
// sums it and updates the row.  In a longer segment every PIECE-th position sums its piece
// into the partial buffer (row index = the piece's first sorted position).
//
// Most segments are short, and for those everything follows from the sorted ids around r alone:
// lane l reads sorted[r - PIECE + l].  Position r opens a segment if sorted[r - 1] differs; the run
// of equal ids from r on is its length if it ends within PIECE positions; a position inside a
// segment and less than PIECE from its start never starts a piece.  So the common case needs the
// ids and the permutation in one round trip to memory and the gradient rows in the next (the table
// row is pulled into L2 meanwhile), instead of a chain through the segment tables; only positions
// in segments longer than PIECE take the general path.
template <typename V, int NCH>
__device__ __forceinline__ void piece_sum(const UpdateJob& J, const UpdateParams& p, int r, int lane) {
    const int wv = J.width / VecOps<V>::LEN;
    {
        const int pos = r - PIECE + lane;
        const int32_t sv = pos < 0 ? -1 : (pos < J.n ? J.sorted[pos] : -2);
        const int32_t after = r + PIECE < J.n ? J.sorted[r + PIECE] : -2;
        const int32_t src = (lane < PIECE && r + lane < J.n) ? J.perm[r + lane] : 0;
        const int32_t id = __shfl_sync(0xffffffffu, sv, PIECE);
        const bool head = __shfl_sync(0xffffffffu, sv, PIECE - 1) != id;
        const bool far = __shfl_sync(0xffffffffu, sv, 0) == id;          // PIECE or more positions into a segment
        const unsigned same = __ballot_sync(0xffffffffu, sv == id) >> PIECE;
        const int run = __ffs(~same) - 1;                                // ids equal to mine from r on, at most PIECE
        if (!head && !far) return;
        if (head && (run < PIECE || after != id)) {
            const int64_t row = id;
            const int row_lines = (J.width * 4 + 127) / 128;
            const char* base = reinterpret_cast<const char*>(J.table + row * J.width);
            if (lane < row_lines) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + lane * 128));
            if (p.opt == KGE_OPT_ADAM) {
                const char* sb = reinterpret_cast<const char*>(J.state + row * 2 * J.width);
                for (int ln = lane; ln < 2 * row_lines; ln += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(sb + ln * 128));
            }
            V g[NCH];
#pragma unroll
            for (int i = 0; i < NCH; ++i) g[i] = VecOps<V>::zero();
            ordered_sum<V, NCH>(reinterpret_cast<const V*>(J.grads), wv, run,
                                [&](int s) { return (int64_t)__shfl_sync(0xffffffffu, src, s); }, g, lane);
            apply_row<V, NCH>(J, p, row, g, lane);
            return;
        }
    }
    const int u = J.seg_of[r];
    const int s0 = J.seg[u], s1 = J.seg[u + 1];
    const int len = s1 - s0;
    const bool whole = len <= PIECE;
    if (whole ? r != s0 : ((r - s0) % PIECE) != 0) return;
    const int count = whole ? len : min(PIECE, s1 - r);
    const int32_t src = lane < count ? J.perm[r + lane] : 0;
    if (whole) {   // start fetching the table row (and its optimiser state) while the gradients are summed
        const int64_t row = J.uniq[u];
        const int row_lines = (J.width * 4 + 127) / 128;
        const char* base = reinterpret_cast<const char*>(J.table + row * J.width);
        if (lane < row_lines) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + lane * 128));
        if (p.opt == KGE_OPT_ADAM) {
            const char* sb = reinterpret_cast<const char*>(J.state + row * 2 * J.width);
            for (int ln = lane; ln < 2 * row_lines; ln += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(sb + ln * 128));
        }
    }
    V g[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) g[i] = VecOps<V>::zero();
    ordered_sum<V, NCH>(reinterpret_cast<const V*>(J.grads), wv, count,
                        [&](int s) { return (int64_t)__shfl_sync(0xffffffffu, src, s); }, g, lane);
    if (whole) {
        apply_row<V, NCH>(J, p, J.uniq[u], g, lane);
        return;
    }
    V* dst = reinterpret_cast<V*>(J.part) + (int64_t)r * wv;
#pragma unroll
    for (int i = 0; i < NCH; ++i) { const int c = lane + 32 * i; if (c < wv) dst[c] = g[i]; }
    // The warp that finishes the segment's last outstanding piece adds all pieces, in ascending
    // order whoever that warp is, and updates the row.
    const int npieces = (len + PIECE - 1) / PIECE;
    __threadfence();
    int done = 0;
    if (lane == 0) done = atomicAdd(&J.seg_done[u], 1);
    done = __shfl_sync(0xffffffffu, done, 0);
    if (done != npieces - 1) return;
    __threadfence();
#pragma unroll
    for (int i = 0; i < NCH; ++i) g[i] = VecOps<V>::zero();
    ordered_sum<V, NCH, true>(reinterpret_cast<const V*>(J.part), wv, npieces,
                              [&](int s) { return (int64_t)s0 + (int64_t)s * PIECE; }, g, lane);
    apply_row<V, NCH>(J, p, J.uniq[u], g, lane);
}

__global__ void __launch_bounds__(256, 4) piece_kernel(UpdateParams p) {
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    grid_dependency_wait();
    if (gw >= p.warp_begin[p.njobs]) return;
    int j = 0;
    while (j + 1 < p.njobs && gw >= p.warp_begin[j + 1]) ++j;
    const UpdateJob& J = p.job[j];
    const int r = gw - p.warp_begin[j];
    if ((J.width & 3) == 0) {
        const int wv = J.width >> 2;
        if (wv <= 32) piece_sum<float4, 1>(J, p, r, lane);
        else if (wv <= 64) piece_sum<float4, 2>(J, p, r, lane);
        else piece_sum<float4, 4>(J, p, r, lane);
    } else {
        // narrow rows whose width is only even (RotatE phases with d % 8 != 0): scalar lanes
        if (J.width <= 64) piece_sum<float, 2>(J, p, r, lane);
        else piece_sum<float, kMaxDim / 2 / 32>(J, p, r, lane);
    }
}

}  // namespace

int dedup_tiles(int n) { return (n + SORT_TILE - 1) / SORT_TILE; }

int launch_dedup(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                 const int32_t* negs, cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg;
    DedupParams dp;
    dp.ent = IdList{heads, tails, negs, B, B, N, c.num_entities,
                    w.ent_perm, w.ent_sorted, w.ent_uniq, w.ent_seg, w.ent_segof, w.ent_done, nullptr, w.ent_tkeys, w.counts};
    dp.rel = IdList{rels, rels, rels, B, 0, 0, c.num_relations,
                    w.rel_perm, w.rel_sorted, w.rel_uniq, w.rel_seg, w.rel_segof, w.rel_done, w.relw_done, w.rel_tkeys, w.counts + 1};
    dp.ent_tiles = dedup_tiles(2 * B + N);
    dp.status = w.status;
    const int tiles = dp.ent_tiles + dedup_tiles(B);
    stage_begin(h, ST_RANK, s);
    tile_sort_kernel<<<tiles, SORT_THREADS, 0, s>>>(dp);
    KGE_LAUNCH_CHECK(h);
    rank_kernel<<<tiles * (SORT_TILE / RANK_THREADS), RANK_THREADS, 0, s>>>(dp);
    stage_end(h, ST_RANK, s);
    KGE_LAUNCH_CHECK(h);
    stage_begin(h, ST_SEGMENT, s);
    segment_kernel<<<2, SEG_THREADS, 0, s>>>(dp);
    stage_end(h, ST_SEGMENT, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

// ---- one list of (row id, gradient row) pairs applied to one table, with caller-provided scratch ----
namespace {
struct ApplyScratch {
    int32_t *perm, *sorted, *uniq, *seg, *segof, *done, *count, *dummy;
    uint64_t* tkeys;
    float* part;
    size_t bytes;
};
// Carves the scratch of a list of n rows of `width` floats (base == nullptr: measures only).
ApplyScratch carve_apply(char* base, int n, int width) {
    size_t used = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + used : nullptr; used += (bytes + 255) / 256 * 256; return p; };
    ApplyScratch a{};
    a.perm = reinterpret_cast<int32_t*>(take((size_t)n * 4)); a.sorted = reinterpret_cast<int32_t*>(take((size_t)n * 4));
    a.uniq = reinterpret_cast<int32_t*>(take((size_t)n * 4)); a.seg = reinterpret_cast<int32_t*>(take(((size_t)n + 1) * 4));
    a.segof = reinterpret_cast<int32_t*>(take((size_t)n * 4)); a.done = reinterpret_cast<int32_t*>(take((size_t)n * 4));
    a.count = reinterpret_cast<int32_t*>(take(256)); a.dummy = reinterpret_cast<int32_t*>(take(256));
    a.tkeys = reinterpret_cast<uint64_t*>(take((size_t)dedup_tiles(n) * SORT_TILE * 8));
    a.part = reinterpret_cast<float*>(take((size_t)n * width * 4));
    a.bytes = used;
    return a;
}
}  // namespace

namespace {
// One warp per requested row: out[i] = table[ids[i] - base] (an id outside the shard is reported and reads row 0).
__global__ void __launch_bounds__(256) gather_rows_kernel(const float* table, int64_t rows, int d4, const int32_t* ids, int n, int64_t base,
                                                          float* out, int32_t* status) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (i >= n) return;
    int64_t r = (int64_t)ids[i] - base;
    if (r < 0 || r >= rows) { set_status(status, KGE_ERR_ID_RANGE); r = 0; }
    const float4* src = reinterpret_cast<const float4*>(table) + r * d4;
    float4* dst = reinterpret_cast<float4*>(out) + (int64_t)i * d4;
    for (int c = lane; c < d4; c += 32) dst[c] = src[c];
}
}  // namespace

int launch_gather_rows(kge_handle* h, const int32_t* ids, int n, int64_t base, float* out, cudaStream_t s) {
    gather_rows_kernel<<<(n * 32 + 255) / 256, 256, 0, s>>>(h->ent, h->cfg.num_entities, h->cfg.dim / 4, ids, n, base, out, h->ws.status);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

size_t apply_scratch_bytes(int n, int width) { return carve_apply(nullptr, n, width).bytes; }

// table[ids[i]] receives the gradient row grads[i] for i < n: stable sort of the ids, one update per distinct row with
// the row's gradients added in ascending list position, by the handle's optimiser rule (the same kernels as the step's
// own update).  `rows`: height of the table; state: the table's optimiser state.
int launch_apply_gradients(kge_handle* h, float* table, float* state, int64_t rows, int width, const int32_t* ids, const float* grads,
                           int n, uint64_t step, float lr, void* scratch, cudaStream_t s) {
    const kge_config& c = h->cfg;
    ApplyScratch a = carve_apply(static_cast<char*>(scratch), n, width);
    DedupParams dp;
    dp.ent = IdList{ids, ids, ids, n, 0, 0, rows, a.perm, a.sorted, a.uniq, a.seg, a.segof, a.done, nullptr, a.tkeys, a.count};
    // (the kernels serve two lists at once: the second one is empty here)
    dp.rel = IdList{ids, ids, ids, 0, 0, 0, rows, a.dummy, a.dummy, a.dummy, a.dummy, a.dummy, a.dummy, nullptr, a.tkeys, a.dummy + 32};
    dp.ent_tiles = dedup_tiles(n);
    dp.status = h->ws.status;
    tile_sort_kernel<<<dp.ent_tiles, SORT_THREADS, 0, s>>>(dp);
    KGE_LAUNCH_CHECK(h);
    rank_kernel<<<dp.ent_tiles * (SORT_TILE / RANK_THREADS), RANK_THREADS, 0, s>>>(dp);
    KGE_LAUNCH_CHECK(h);
    segment_kernel<<<2, SEG_THREADS, 0, s>>>(dp);
    KGE_LAUNCH_CHECK(h);
    UpdateParams up;
    up.njobs = 1;
    up.job[0] = UpdateJob{table, state, grads, a.part, a.uniq, a.seg, a.perm, a.sorted, a.segof, a.done, width, n};
    up.job[1] = up.job[0]; up.job[2] = up.job[0];
    up.warp_begin[0] = 0; up.warp_begin[1] = n; up.warp_begin[2] = n; up.warp_begin[3] = n;
    up.opt = c.opt;
    up.lr = lr; up.beta1 = c.beta1; up.beta2 = c.beta2; up.eps = c.eps;
    up.corr1 = (float)(1.0 - std::pow((double)c.beta1, (double)(step + 1)));
    up.corr2 = (float)(1.0 - std::pow((double)c.beta2, (double)(step + 1)));
    KGE_CUDA_CHECK(h, launch_dependent(piece_kernel, dim3((n * 32 + 255) / 256), dim3(256), 0, s, up));
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

int launch_update(kge_handle* h, uint64_t step, float lr, cudaStream_t s) {
    const kge_config& c = h->cfg;
    Workspace& w = h->ws;
    const int B = c.batch, N = c.num_neg;
    UpdateParams up;
    up.njobs = c.score == KGE_TRANSH ? 3 : 2;
    up.job[0] = UpdateJob{h->ent, h->ent_state, w.grad_ent, w.part_ent, w.ent_uniq, w.ent_seg, w.ent_perm,
                          w.ent_sorted, w.ent_segof, w.ent_done, c.dim, 2 * B + N};
    up.job[1] = UpdateJob{h->rel, h->rel_state, w.grad_rel, w.part_rel, w.rel_uniq, w.rel_seg, w.rel_perm,
                          w.rel_sorted, w.rel_segof, w.rel_done, h->kw, B};
    up.job[2] = UpdateJob{h->relw, h->relw_state, w.grad_relw, w.part_relw, w.rel_uniq, w.rel_seg, w.rel_perm,
                          w.rel_sorted, w.rel_segof, w.relw_done, c.dim, B};
    up.warp_begin[0] = 0;
    for (int j = 0; j < 3; ++j) up.warp_begin[j + 1] = up.warp_begin[j] + (j < up.njobs ? up.job[j].n : 0);
    up.opt = c.opt;
    up.lr = lr; up.beta1 = c.beta1; up.beta2 = c.beta2; up.eps = c.eps;
    up.corr1 = (float)(1.0 - std::pow((double)c.beta1, (double)(step + 1)));
    up.corr2 = (float)(1.0 - std::pow((double)c.beta2, (double)(step + 1)));
    const int warps = up.warp_begin[up.njobs];
    stage_begin(h, ST_UPDATE, s);
    KGE_CUDA_CHECK(h, launch_dependent(piece_kernel, dim3((warps * 32 + 255) / 256), dim3(256), 0, s, up));
    stage_end(h, ST_UPDATE, s);
    KGE_LAUNCH_CHECK(h);
    return KGE_OK;
}

}  // namespace kge
