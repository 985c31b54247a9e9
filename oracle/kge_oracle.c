/*
 * kge_oracle.c -- CPU oracle for the shared-negative scoring block of BESS-style
 * knowledge-graph-embedding training and inference.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the plain, slow, definition-level
 * statement of what the hot path computes, written from the paper, and it is
 * what the CUDA library is checked against.  Only the tests, the smoke check and
 * the benchmark's "cpu_baseline"/"reference" legs may call it; the product never
 * does.  It shares no source, header, table or helper with the CUDA library.
 *
 * Precision: compiled twice from this one source.
 *   -DKGEO_F32=0 (default)  real = double : the truth for every tolerance check
 *                                           and for finite differences.
 *   -DKGEO_F32=1            real = float  : used only where floating point decides
 *                                           an integer (top-k ids, ranks), so that
 *                                           oracle and kernel decide in the same
 *                                           precision.  Its arithmetic order per
 *                                           pair is: index k ascending, a single
 *                                           accumulator, fused multiply-add exactly
 *                                           where fma() is written below.
 * Compile with -O2 -fno-fast-math -ffp-contract=off so that nothing is fused or
 * reassociated beyond what is written.
 *
 * Sub-gradient of |x| at x = 0 (p = 1 distances): 0 by default.  Any value in [-1, 1] is a valid
 * sub-gradient there; a third build with -DKGEO_L1_TIE_SIGN=-1 takes sign(0) = -1 (the left
 * derivative) and exists only so that a test on constructed exact ties can check, coordinate by
 * coordinate, which sub-gradient the CUDA library takes.  It differs from the default build at
 * exact ties only (pinned by a closed form on TransE).
 *
 * Parity pins (tests/test_oracle_*.py, all CPU):
 *   philox4x32_10      : cross-checked against cuRAND's host Philox generator.
 *   mulhi64, icbrt     : Python big-integer arithmetic.
 *   init_table         : moments and Kolmogorov-Smirnov tests against the normal / uniform laws,
 *                        independence of neighbouring entries, the raw words against philox.
 *   graph_build        : brute-force bucket membership + stable order on tiny graphs.
 *   sample_batch       : exact per-bucket / per-partition counts (Eq. 3, Eq. 4),
 *                        chi-square of the cube-root relation law.
 *   bf16_round         : hand-worked IEEE bit patterns (ties to even both ways, carries,
 *                        negatives, subnormals, the largest finite value) and an independent
 *                        rounding routine on 10^5 random floats.
 *   query_vector       : numpy restatement per model; f(h, r, t) recovered from (q, t) alone.
 *   score              : TransE 0 at h=t,r=0; DistMult symmetry; ComplEx -> DistMult
 *                        with zero imaginary parts; RotatE zero phase -> complex L1;
 *                        TransH special cases; numpy.linalg.norm for the L2 forms.
 *   batch_loss         : closed forms (log(N+1), log|E|, 2 log 2), softmax sums to 1.
 *   batch_grads        : central finite differences of batch_loss in fp64 (also with the
 *                        L3 regulariser switched on, both forms).
 *   l3_term            : hand values (1, -2, 2) -> 17^(1/3) and 17; homogeneity.
 *   lr_linear_decay    : end points, midpoint, linearity.
 *   encoder_*          : e = e_S + M e_F against numpy for one slot; central finite differences of the
 *                        encoder batch loss in every coordinate of M_H, M_T and the shallow rows; the
 *                        shared-matrix step against the sum of the two gradients.
 *   ensemble_topk      : a hand-worked 3-model example (p = -0.5, p = 1), reciprocal-rank fusion (p = -1)
 *                        restated in numpy, invariance under a permutation of the models, the id tie rule.
 *   dedup/update_rows  : naive scatter when all ids differ; hand sums when they repeat;
 *                        independent numpy restatement of an SGD step.
 *   score_all_topk     : numpy argsort brute force; duplicated rows (exact ties).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef KGEO_F32
#define KGEO_F32 0
#endif
#ifndef KGEO_L1_TIE_SIGN
#define KGEO_L1_TIE_SIGN 0
#endif

#if KGEO_F32
typedef float real;
#define R_SQRT sqrtf
#define R_EXP expf
#define R_LOG logf
#define R_LOG1P log1pf
#define R_FABS fabsf
#define R_FMA fmaf
#define R_SIN sinf
#define R_COS cosf
#else
typedef double real;
#define R_SQRT sqrt
#define R_EXP exp
#define R_LOG log
#define R_LOG1P log1p
#define R_FABS fabs
#define R_FMA fma
#define R_SIN sin
#define R_COS cos
#endif

enum { SC_TRANSE = 0, SC_TRANSH = 1, SC_ROTATE = 2, SC_DISTMULT = 3, SC_COMPLEX = 4,
       SC_ROTATE_REAL = 5 };   /* RotatE with the norm taken literally over the d real coordinates (see distance_norm) */
static int is_rotate(int32_t score) { return score == SC_ROTATE || score == SC_ROTATE_REAL; }
enum { LOSS_LOGSIGMOID = 0, LOSS_SAMPLED_SOFTMAX = 1 };
enum { OPT_SGD = 0, OPT_ADAM = 1, OPT_ROWWISE_ADAGRAD = 2 };
enum { ERR_OK = 0, ERR_BAD_ARG = -1, ERR_DIVISIBILITY = -2, ERR_EMPTY_BUCKET = -3 };

/* All floating-point hyper-parameters are doubles whatever `real` is. */
typedef struct {
    int64_t num_entities, num_relations;
    int32_t dim;           /* real numbers per entity row (even for RotatE / ComplEx) */
    int32_t score;         /* SC_* */
    int32_t p_norm;        /* 1 or 2 (distance models) */
    int32_t loss;          /* LOSS_* */
    int32_t opt;           /* OPT_* */
    int32_t bf16_operands; /* 1: block scores of dot-product models and TransE-L2 use
                              bf16-rounded query/tail operands (tensor-core variant) */
    int32_t batch, num_neg, num_parts;
    int32_t head_part;     /* -1: slots spread over all P*P buckets; i: micro-batch B_i */
    int32_t sample_mode;   /* 0: cube-root relation law; 1: uniform over the bucket */
    int32_t bf16_projection; /* 1: the encoder's projection M e_F takes M rounded to bf16 (tensor-core variant) */
    double gamma, adv_temp, ce_correction, loss_scale;
    double lr, beta1, beta2, eps;
    uint64_t seed;
    double reg_lambda;     /* lambda_S of the L3 regulariser on the gathered entity rows (0 = off) */
    int32_t reg_form;      /* 0: sum of the norms ||e||_3 as printed; 1: sum of the cubes ||e||_3^3 */
    int32_t _pad2;
} kgeo_config;

int kgeo_real_bytes(void) { return (int)sizeof(real); }

/* ------------------------------------------------------------------------- */
/* Counter-based random numbers: Philox4x32 with 10 rounds (Salmon, Moraes,   */
/* Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11).         */
/* ------------------------------------------------------------------------- */
void kgeo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* floor(a * n / 2^64): maps a uniform 64-bit word onto [0, n). */
uint64_t kgeo_mulhi64(uint64_t a, uint64_t n) {
    return (uint64_t)(((unsigned __int128)a * (unsigned __int128)n) >> 64);
}

/* Two 64-bit words for (slot, step, stream) under `seed`. */
static void draw2x64(uint64_t seed, uint64_t step, uint32_t slot, uint32_t stream,
                     uint64_t *x64, uint64_t *y64) {
    uint32_t ctr[4] = { slot, (uint32_t)step, (uint32_t)(step >> 32), stream };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t o[4];
    kgeo_philox4x32_10(ctr, key, o);
    *x64 = (uint64_t)o[0] | ((uint64_t)o[1] << 32);
    *y64 = (uint64_t)o[2] | ((uint64_t)o[3] << 32);
}

/* ------------------------------------------------------------------------- */
/* Table initialisation.  The paper prescribes none; this is the library's     */
/* recipe: element (row, 4c + j) of a [rows, width] table comes from word j of  */
/* Philox with counter (row lo, row hi, c, stream) under the seed, through the   */
/* uniform u = ((word >> 9) + 1/2) 2^-23 in (0, 1).  kind 0: normal entries by   */
/* Box-Muller on the word pairs (0, 1) and (2, 3): std sqrt(-2 ln u_a) times      */
/* (cos, sin)(2 pi u_b).  kind 1: phases (2u - 1) pi.  kind 2: the raw words      */
/* (as bit patterns).  Computed in fp64, stored as fp32 like every table.         */
/* ------------------------------------------------------------------------- */
void kgeo_init_table(uint64_t seed, uint32_t stream, int64_t rows, int32_t width, double std,
                     int32_t kind, float *out) {
    const double PI = 3.14159265358979323846;
    for (int64_t row = 0; row < rows; ++row) {
        for (int32_t c = 0; 4 * c < width; ++c) {
            uint32_t ctr[4] = { (uint32_t)row, (uint32_t)((uint64_t)row >> 32), (uint32_t)c, stream };
            uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
            uint32_t x[4];
            kgeo_philox4x32_10(ctr, key, x);
            double u[4], v[4];
            for (int j = 0; j < 4; ++j) u[j] = ((double)(x[j] >> 9) + 0.5) / 8388608.0;
            if (kind == 1) {
                for (int j = 0; j < 4; ++j) v[j] = (2.0 * u[j] - 1.0) * PI;
            } else {
                for (int j = 0; j < 4; j += 2) {
                    double rad = std * sqrt(-2.0 * log(u[j]));
                    v[j] = rad * cos(2.0 * PI * u[j + 1]);
                    v[j + 1] = rad * sin(2.0 * PI * u[j + 1]);
                }
            }
            for (int j = 0; j < 4 && 4 * c + j < width; ++j) {
                float f = (float)v[j];
                if (kind == 2) memcpy(&f, &x[j], 4);
                out[row * width + 4 * c + j] = f;
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Partitions, buckets, cube-root weights (Section 4, "Partitioning" and      */
/* "Training": T_{i,j}, n_r counted inside the bucket, p(r) ~ n_r^(1/3)).     */
/* ------------------------------------------------------------------------- */

/* Integer cube-root weight: the largest w with w^3 <= n * 2^60 (0 for n = 0).
 * Integer weights make the sampling law bit-reproducible on any machine. */
uint64_t kgeo_icbrt_weight(uint64_t n) {
    if (n == 0) return 0;
    unsigned __int128 target = (unsigned __int128)n << 60;
    uint64_t lo = 0, hi = (uint64_t)1 << 42; /* (2^64 * 2^60)^(1/3) < 2^42 */
    while (lo < hi) { /* invariant: lo^3 <= target < (hi+1)^3 */
        uint64_t mid = lo + (hi - lo + 1) / 2;
        unsigned __int128 cube = (unsigned __int128)mid * mid * mid;
        if (cube <= target) lo = mid; else hi = mid - 1;
    }
    return lo;
}

static int64_t shard_size(int64_t E, int32_t P) { return (E + P - 1) / P; }

/*
 * Canonical triple order = STABLE sort of the caller's list by (part(h), part(t), r),
 * part(e) = e div ceil(E/P).  off[(i*P+j)*(R+1)+r] = first sorted index of relation r
 * in bucket (i,j) (entry R = end of the bucket); wcum = running sum of the integer
 * cube-root weights inside the bucket (entry 0 = 0, entry R = bucket total).
 */
int kgeo_graph_build(int64_t E, int64_t R, int32_t P, int64_t T,
                     const int32_t *h, const int32_t *r, const int32_t *t,
                     int32_t *sh, int32_t *sr, int32_t *st,
                     int64_t *off, uint64_t *wcum) {
    if (E <= 0 || R <= 0 || P <= 0 || T < 0) return ERR_BAD_ARG;
    int64_t S = shard_size(E, P);
    int64_t nkeys = (int64_t)P * P * R;
    int64_t *count = (int64_t *)calloc((size_t)nkeys + 1, sizeof(int64_t));
    if (!count) return ERR_BAD_ARG;
    for (int64_t e = 0; e < T; ++e) {
        if (h[e] < 0 || h[e] >= E || t[e] < 0 || t[e] >= E || r[e] < 0 || r[e] >= R) {
            free(count); return ERR_BAD_ARG;
        }
        int64_t key = ((h[e] / S) * P + (t[e] / S)) * R + r[e];
        count[key + 1] += 1;
    }
    for (int64_t k = 0; k < nkeys; ++k) count[k + 1] += count[k]; /* count[k] = start of key k */
    for (int64_t b = 0; b < (int64_t)P * P; ++b) {
        uint64_t acc = 0;
        for (int64_t rr = 0; rr <= R; ++rr) {
            off[b * (R + 1) + rr] = count[b * R + rr]; /* rr = R reads the next bucket's start */
            wcum[b * (R + 1) + rr] = acc;
            if (rr < R) acc += kgeo_icbrt_weight((uint64_t)(count[b * R + rr + 1] - count[b * R + rr]));
        }
    }
    /* stable placement: walk the input in order, append to the key's run */
    int64_t *cursor = (int64_t *)malloc((size_t)nkeys * sizeof(int64_t));
    if (!cursor) { free(count); return ERR_BAD_ARG; }
    memcpy(cursor, count, (size_t)nkeys * sizeof(int64_t));
    for (int64_t e = 0; e < T; ++e) {
        int64_t key = ((h[e] / S) * P + (t[e] / S)) * R + r[e];
        int64_t dst = cursor[key]++;
        sh[dst] = h[e]; sr[dst] = r[e]; st[dst] = t[e];
    }
    free(cursor); free(count);
    return ERR_OK;
}

/*
 * One batch: B positive triples (Eq. 3, with the cube-root relation law) and N shared
 * negative tails (Eq. 4).  Everything is drawn with replacement.
 */
int kgeo_sample_batch(const kgeo_config *c, uint64_t step,
                      const int32_t *sh, const int32_t *sr, const int32_t *st,
                      const int64_t *off, const uint64_t *wcum,
                      int32_t *heads, int32_t *rels, int32_t *tails, int32_t *negs) {
    const int64_t E = c->num_entities, R = c->num_relations;
    const int32_t P = c->num_parts, B = c->batch, N = c->num_neg;
    if (P <= 0 || B <= 0 || N <= 0) return ERR_BAD_ARG;
    if (N % P != 0) return ERR_DIVISIBILITY;
    if (c->head_part < 0 ? (B % (P * P) != 0) : (B % P != 0)) return ERR_DIVISIBILITY;
    if (c->head_part >= P) return ERR_BAD_ARG;
    const int64_t S = shard_size(E, P);
    for (int32_t s = 0; s < B; ++s) {
        int32_t i, j;
        if (c->head_part < 0) { /* all P*P buckets, B/P^2 slots each, bucket-major */
            int32_t beta = s / (B / (P * P));
            i = beta / P; j = beta % P;
        } else {                /* the paper's micro-batch B_i: B/P slots per tail partition */
            i = c->head_part; j = s / (B / P);
        }
        const int64_t base = ((int64_t)i * P + j) * (R + 1);
        uint64_t x64, y64;
        draw2x64(c->seed, step, (uint32_t)s, 0u, &x64, &y64);
        int64_t idx;
        if (c->sample_mode == 0) {
            uint64_t W = wcum[base + R];
            if (W == 0) return ERR_EMPTY_BUCKET;
            uint64_t u = kgeo_mulhi64(x64, W);
            int64_t rr = 0;            /* the unique rr with wcum[rr] <= u < wcum[rr+1] */
            while (!(wcum[base + rr] <= u && u < wcum[base + rr + 1])) ++rr;
            uint64_t n_r = (uint64_t)(off[base + rr + 1] - off[base + rr]);
            idx = off[base + rr] + (int64_t)kgeo_mulhi64(y64, n_r);
        } else {
            uint64_t n_b = (uint64_t)(off[base + R] - off[base]);
            if (n_b == 0) return ERR_EMPTY_BUCKET;
            idx = off[base] + (int64_t)kgeo_mulhi64(x64, n_b);
        }
        heads[s] = sh[idx]; rels[s] = sr[idx]; tails[s] = st[idx];
    }
    for (int32_t n = 0; n < N; ++n) { /* N/P uniform entities from each partition E_j */
        int32_t j = n / (N / P);
        int64_t size_j = E - (int64_t)j * S; if (size_j > S) size_j = S;
        if (size_j <= 0) return ERR_EMPTY_BUCKET;
        uint64_t x64, y64;
        draw2x64(c->seed, step, (uint32_t)n, 1u, &x64, &y64);
        negs[n] = (int32_t)((int64_t)j * S + (int64_t)kgeo_mulhi64(x64, (uint64_t)size_j));
    }
    return ERR_OK;
}

/* ------------------------------------------------------------------------- */
/* Scoring functions (Table "Scoring functions").  One triple at a time, from  */
/* the raw rows.  Complex rows are interleaved (re0, im0, re1, im1, ...).      */
/* RotatE's L1 is the sum of complex moduli (the cited RotatE definition).     */
/* ------------------------------------------------------------------------- */
static int rel_width(int32_t score, int32_t d) { return is_rotate(score) ? d / 2 : d; }

static real bf16_round(real v) { /* round-to-nearest-even to 8 significand bits */
    float f = (float)v;
    uint32_t u; memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return v; /* inf / nan untouched */
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return (real)f;
}

/* The operand rounding of the tensor-core variant, exported so that it can be pinned on bit patterns. */
real kgeo_bf16_round(real v) { return bf16_round(v); }

/* TransH unit normal: w / max(||w||_2, 1e-12). */
static real unit_normal(int32_t d, const real *w, real *what) {
    real s = 0;
    for (int k = 0; k < d; ++k) s = R_FMA(w[k], w[k], s);
    real nrm = R_SQRT(s);
    real den = nrm > (real)1e-12 ? nrm : (real)1e-12;
    for (int k = 0; k < d; ++k) what[k] = w[k] / den;
    return den;
}

/* Residual x of the three distance models, x in R^d (RotatE: interleaved complex). */
static void distance_residual(int32_t score, int32_t d, const real *h, const real *r,
                              const real *what, const real *t, real *x) {
    if (score == SC_TRANSE) {
        for (int k = 0; k < d; ++k) x[k] = (h[k] + r[k]) - t[k];
    } else if (score == SC_TRANSH) {
        /* (h - (w.h) w) + r - (t - (w.t) w) */
        real a = 0, u = 0;
        for (int k = 0; k < d; ++k) a = R_FMA(what[k], h[k], a);
        for (int k = 0; k < d; ++k) u = R_FMA(what[k], t[k], u);
        for (int k = 0; k < d; ++k) {
            real q = R_FMA(-a, what[k], h[k]) + r[k];
            x[k] = R_FMA(u, what[k], q - t[k]);
        }
    } else { /* RotatE: h o e^{i r} - t */
        for (int k = 0; k < d / 2; ++k) {
            real cs = R_COS(r[k]), sn = R_SIN(r[k]);
            real qre = R_FMA(h[2 * k], cs, -(h[2 * k + 1] * sn));
            real qim = R_FMA(h[2 * k], sn, h[2 * k + 1] * cs);
            x[2 * k] = qre - t[2 * k];
            x[2 * k + 1] = qim - t[2 * k + 1];
        }
    }
}

static real distance_norm(int32_t score, int32_t p, int32_t d, const real *x) {
    real acc = 0;
    if (p == 2) {
        for (int k = 0; k < d; ++k) acc = R_FMA(x[k], x[k], acc);
        return R_SQRT(acc);
    }
    if (score == SC_ROTATE) {
        for (int k = 0; k < d / 2; ++k)
            acc += R_SQRT(R_FMA(x[2 * k], x[2 * k], x[2 * k + 1] * x[2 * k + 1]));
        return acc;
    }
    for (int k = 0; k < d; ++k) acc += R_FABS(x[k]);
    return acc;
}

/* Query vector of the two dot-product models: DistMult r o h, ComplEx r * h. */
static void dot_query(int32_t score, int32_t d, const real *h, const real *r, real *q) {
    if (score == SC_DISTMULT) {
        for (int k = 0; k < d; ++k) q[k] = r[k] * h[k];
    } else {
        for (int k = 0; k < d / 2; ++k) {
            q[2 * k] = R_FMA(r[2 * k], h[2 * k], -(r[2 * k + 1] * h[2 * k + 1]));
            q[2 * k + 1] = R_FMA(r[2 * k], h[2 * k + 1], r[2 * k + 1] * h[2 * k]);
        }
    }
}

/*
 * Per-query vector q of the scoring-function table, the part of f(h, r, t) that does not depend
 * on the tail: TransE h + r; TransH (h - (w^.h) w^) + r with w^ the unit normal; RotatE h o e^{i r};
 * DistMult r o h; ComplEx r h.  The score is then a function of (q, t) (and w^ for TransH).
 */
void kgeo_query_vector(int32_t score, int32_t d, const real *h, const real *r, const real *w, real *q) {
    if (score == SC_DISTMULT || score == SC_COMPLEX) { dot_query(score, d, h, r, q); return; }
    if (score == SC_TRANSE) { for (int k = 0; k < d; ++k) q[k] = h[k] + r[k]; return; }
    if (is_rotate(score)) {
        for (int k = 0; k < d / 2; ++k) {
            real cs = R_COS(r[k]), sn = R_SIN(r[k]);
            q[2 * k] = R_FMA(h[2 * k], cs, -(h[2 * k + 1] * sn));
            q[2 * k + 1] = R_FMA(h[2 * k], sn, h[2 * k + 1] * cs);
        }
        return;
    }
    real *what = (real *)malloc(sizeof(real) * (size_t)d);
    unit_normal(d, w, what);
    real a = 0;
    for (int k = 0; k < d; ++k) a = R_FMA(what[k], h[k], a);
    for (int k = 0; k < d; ++k) q[k] = R_FMA(-a, what[k], h[k]) + r[k];
    free(what);
}

/*
 * f(h, r, t).  `w` is the TransH normal (ignored otherwise); `scratch` holds 3*d reals.
 * bf16 = 1 rounds the two operands of the contraction to bf16 first (dot-product
 * models: q and t; TransE-L2: q = h + r and t inside the cross term only).
 */
static real score_one(int32_t score, int32_t p, int32_t d, int bf16,
                      const real *h, const real *r, const real *w, const real *t, real *scratch) {
    real *x = scratch, *what = scratch + d;
    if (score == SC_DISTMULT || score == SC_COMPLEX) {
        dot_query(score, d, h, r, x);
        real acc = 0;
        if (bf16) for (int k = 0; k < d; ++k) acc = R_FMA(bf16_round(x[k]), bf16_round(t[k]), acc);
        else      for (int k = 0; k < d; ++k) acc = R_FMA(x[k], t[k], acc);
        return acc;
    }
    if (bf16 && score == SC_TRANSE && p == 2) {
        /* ||q||^2 + ||t||^2 - 2 q.t with only the cross term in bf16, clamped at 0 */
        real qq = 0, tt = 0, qt = 0;
        for (int k = 0; k < d; ++k) {
            real q = h[k] + r[k];
            qq = R_FMA(q, q, qq); tt = R_FMA(t[k], t[k], tt);
            qt = R_FMA(bf16_round(q), bf16_round(t[k]), qt);
        }
        real d2 = qq + tt - 2 * qt;
        return -R_SQRT(d2 > 0 ? d2 : 0);
    }
    if (score == SC_TRANSH) unit_normal(d, w, what);
    distance_residual(score, d, h, r, what, t, x);
    return -distance_norm(score, p, d, x);
}

real kgeo_score(int32_t score, int32_t p, int32_t d, int32_t bf16,
                const real *h, const real *r, const real *w, const real *t) {
    real *scratch = (real *)malloc(sizeof(real) * 3 * (size_t)d);
    real f = score_one(score, p, d, bf16, h, r, w, t, scratch);
    free(scratch);
    return f;
}

/*
 * Accumulate g * df/d(h, r, w, t) into dh, dr, dw, dt (any of which may be NULL).
 * Exact derivatives of the definitions above (never of the bf16 variant);
 * conventions at the kinks: sign(0) = 0, zero gradient at zero distance / modulus.
 * `scratch` holds 6*d reals.
 */
static void score_grad_one(int32_t score, int32_t p, int32_t d, real g,
                           const real *h, const real *r, const real *w, const real *t,
                           real *dh, real *dr, real *dw, real *dt, real *scratch) {
    real *x = scratch, *what = scratch + d, *s = scratch + 2 * d, *dwhat = scratch + 3 * d;
    if (score == SC_DISTMULT) {
        for (int k = 0; k < d; ++k) {
            if (dh) dh[k] += g * r[k] * t[k];
            if (dr) dr[k] += g * h[k] * t[k];
            if (dt) dt[k] += g * r[k] * h[k];
        }
        return;
    }
    if (score == SC_COMPLEX) { /* f = Re sum r h conj(t) */
        for (int k = 0; k < d / 2; ++k) {
            real hr = h[2 * k], hi = h[2 * k + 1], rr = r[2 * k], ri = r[2 * k + 1];
            real tr = t[2 * k], ti = t[2 * k + 1];
            /* f_k = (rr hr - ri hi) tr + (rr hi + ri hr) ti */
            if (dh) { dh[2 * k] += g * (rr * tr + ri * ti); dh[2 * k + 1] += g * (-ri * tr + rr * ti); }
            if (dr) { dr[2 * k] += g * (hr * tr + hi * ti); dr[2 * k + 1] += g * (-hi * tr + hr * ti); }
            if (dt) { dt[2 * k] += g * (rr * hr - ri * hi); dt[2 * k + 1] += g * (rr * hi + ri * hr); }
        }
        return;
    }
    real den = 1;
    if (score == SC_TRANSH) den = unit_normal(d, w, what);
    distance_residual(score, d, h, r, what, t, x);
    /* s = df/dx, f = -norm(x) */
    if (p == 2) {
        real nrm = distance_norm(score, 2, d, x);
        for (int k = 0; k < d; ++k) s[k] = nrm > 0 ? -x[k] / nrm : 0;
    } else if (score == SC_ROTATE) {
        for (int k = 0; k < d / 2; ++k) {
            real m = R_SQRT(x[2 * k] * x[2 * k] + x[2 * k + 1] * x[2 * k + 1]);
            s[2 * k] = m > 0 ? -x[2 * k] / m : 0;
            s[2 * k + 1] = m > 0 ? -x[2 * k + 1] / m : 0;
        }
    } else {
        for (int k = 0; k < d; ++k) s[k] = x[k] > 0 ? (real)-1 : (x[k] < 0 ? (real)1 : -(real)KGEO_L1_TIE_SIGN);
    }
    if (score == SC_TRANSE) { /* x = h + r - t */
        for (int k = 0; k < d; ++k) {
            if (dh) dh[k] += g * s[k];
            if (dr) dr[k] += g * s[k];
            if (dt) dt[k] -= g * s[k];
        }
    } else if (is_rotate(score)) { /* x = h e^{i theta} - t */
        for (int k = 0; k < d / 2; ++k) {
            real cs = R_COS(r[k]), sn = R_SIN(r[k]);
            real sre = s[2 * k], sim = s[2 * k + 1];
            real qre = h[2 * k] * cs - h[2 * k + 1] * sn, qim = h[2 * k] * sn + h[2 * k + 1] * cs;
            if (dh) { dh[2 * k] += g * (sre * cs + sim * sn); dh[2 * k + 1] += g * (-sre * sn + sim * cs); }
            if (dr) dr[k] += g * (-sre * qim + sim * qre);
            if (dt) { dt[2 * k] -= g * sre; dt[2 * k + 1] -= g * sim; }
        }
    } else { /* TransH: x = delta + r - (what.delta) what, delta = h - t */
        real ws = 0, wdelta = 0;
        for (int k = 0; k < d; ++k) { ws += what[k] * s[k]; wdelta += what[k] * (h[k] - t[k]); }
        for (int k = 0; k < d; ++k) {
            real ddelta = s[k] - ws * what[k];
            if (dh) dh[k] += g * ddelta;
            if (dt) dt[k] -= g * ddelta;
            if (dr) dr[k] += g * s[k];
            dwhat[k] = -(h[k] - t[k]) * ws - wdelta * s[k];
        }
        if (dw) { /* through what = w / den */
            real wd = 0, nrm2 = 0;
            for (int k = 0; k < d; ++k) { wd += what[k] * dwhat[k]; nrm2 += w[k] * w[k]; }
            int clamped = !(R_SQRT(nrm2) > (real)1e-12);
            for (int k = 0; k < d; ++k)
                dw[k] += g * (clamped ? dwhat[k] / den : (dwhat[k] - wd * what[k]) / den);
        }
    }
}

void kgeo_score_grad(int32_t score, int32_t p, int32_t d, real g,
                     const real *h, const real *r, const real *w, const real *t,
                     real *dh, real *dr, real *dw, real *dt) {
    real *scratch = (real *)malloc(sizeof(real) * 6 * (size_t)d);
    score_grad_one(score, p, d, g, h, r, w, t, dh, dr, dw, dt, scratch);
    free(scratch);
}

/* ------------------------------------------------------------------------- */
/* Losses (Section 3.1 "Loss Functions").                                      */
/* ------------------------------------------------------------------------- */
static real softplus(real z) { return (z > 0 ? z : 0) + R_LOG1P(R_EXP(-R_FABS(z))); }
static real sigmoid(real z) {
    if (z >= 0) return 1 / (1 + R_EXP(-z));
    real e = R_EXP(z); return e / (1 + e);
}

/*
 * Loss of one positive with score fpos against N negative scores F[0..N).
 * Writes dL/dfpos to *gpos and dL/dF[n] to G[n] (before loss_scale).
 * Log-sigmoid: -log sig(gamma + f+) - sum_n w_n log sig(-gamma - F_n),
 *   w = softmax_n(a F) held constant in the derivative (StopGrad); `w_fixed`, when
 *   given, replaces the softmax (used by the finite-difference pin).
 * Sampled softmax: -f+ + log(exp f+ + sum_n exp(F_n + c)).
 */
static real row_loss(const kgeo_config *c, real fpos, const real *F, int32_t N,
                     const real *w_fixed, real *gpos, real *G) {
    if (c->loss == LOSS_LOGSIGMOID) {
        const real gamma = (real)c->gamma, a = (real)c->adv_temp;
        real m = a * F[0];
        for (int n = 1; n < N; ++n) if (a * F[n] > m) m = a * F[n];
        real z = 0;
        for (int n = 0; n < N; ++n) z += R_EXP(a * F[n] - m);
        real L = softplus(-(gamma + fpos));
        if (gpos) *gpos = -sigmoid(-(gamma + fpos));
        for (int n = 0; n < N; ++n) {
            real wn = w_fixed ? w_fixed[n] : R_EXP(a * F[n] - m) / z;
            L += wn * softplus(gamma + F[n]);
            if (G) G[n] = wn * sigmoid(gamma + F[n]);
        }
        return L;
    } else {
        const real cc = (real)c->ce_correction;
        real m = fpos;
        for (int n = 0; n < N; ++n) if (F[n] + cc > m) m = F[n] + cc;
        real z = R_EXP(fpos - m);
        for (int n = 0; n < N; ++n) z += R_EXP(F[n] + cc - m);
        if (gpos) *gpos = R_EXP(fpos - m) / z - 1;
        if (G) for (int n = 0; n < N; ++n) G[n] = R_EXP(F[n] + cc - m) / z;
        return -fpos + (m + R_LOG(z));
    }
}

real kgeo_row_loss(const kgeo_config *c, real fpos, const real *F, int32_t N,
                   const real *w_fixed, real *gpos, real *G) {
    return row_loss(c, fpos, F, N, w_fixed, gpos, G);
}

/* ------------------------------------------------------------------------- */
/* Regularisation (Section 3.1 "Regularisation"): lambda_S Omega_S with          */
/* Omega_S = sum over the batch of (||h||_3 + ||t||_3) + sum over the shared     */
/* negatives of ||t'||_3, one term per occurrence of a row.  There is no feature  */
/* projection here, so the final embedding is the shallow one and Omega_T equals  */
/* Omega_S.  The term is added to the micro-batch loss as it stands (it is not    */
/* multiplied by loss_scale).  reg_form 1 takes the cube of each norm instead     */
/* (the form of the regulariser's source, Lacroix et al. 2018).                   */
/* ------------------------------------------------------------------------- */
real kgeo_l3_term(int32_t form, int32_t d, const real *e) {
    real s3 = 0;
    for (int k = 0; k < d; ++k) s3 += R_FABS(e[k]) * e[k] * e[k];
    return form == 1 ? s3 : (real)cbrt((double)s3);
}

/* g[k] += lam * d(term)/d e[k]; the norm has zero gradient at e = 0. */
static void l3_term_grad(int32_t form, int32_t d, real lam, const real *e, real *g) {
    real s3 = 0;
    for (int k = 0; k < d; ++k) s3 += R_FABS(e[k]) * e[k] * e[k];
    if (form == 1) { for (int k = 0; k < d; ++k) g[k] += lam * 3 * e[k] * R_FABS(e[k]); return; }
    if (!(s3 > 0)) return;
    real n = (real)cbrt((double)s3);
    for (int k = 0; k < d; ++k) g[k] += lam * e[k] * R_FABS(e[k]) / (n * n);
}

static double batch_regulariser(const kgeo_config *c, const real *ent, const int32_t *heads,
                                const int32_t *tails, const int32_t *negs) {
    if (c->reg_lambda == 0) return 0;
    const int32_t d = c->dim;
    double omega = 0;
    for (int32_t b = 0; b < c->batch; ++b)
        omega += (double)kgeo_l3_term(c->reg_form, d, ent + (size_t)heads[b] * d)
               + (double)kgeo_l3_term(c->reg_form, d, ent + (size_t)tails[b] * d);
    for (int32_t n = 0; n < c->num_neg; ++n) omega += (double)kgeo_l3_term(c->reg_form, d, ent + (size_t)negs[n] * d);
    return c->reg_lambda * omega;
}

static const real *relw_row(const real *relw, int64_t r, int32_t d) {
    return relw ? relw + (size_t)r * d : NULL;
}

/*
 * Forward of one batch: fpos[B], F[B,N] (row-major), per-row loss Lrow[B] (any may be
 * NULL), returns loss_scale * sum_b L_b.  w_fixed: optional [B,N] constant weights.
 */
double kgeo_batch_loss(const kgeo_config *c, const real *ent, const real *rel, const real *relw,
                       const int32_t *heads, const int32_t *rels, const int32_t *tails,
                       const int32_t *negs, const real *w_fixed,
                       real *fpos_out, real *F_out, real *Lrow_out) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    const int kw = rel_width(c->score, d);
    double total = 0;
    real *Lrow = (real *)malloc(sizeof(real) * (size_t)B);
#pragma omp parallel
    {
        real *scratch = (real *)malloc(sizeof(real) * 3 * (size_t)d);
        real *Frow = (real *)malloc(sizeof(real) * (size_t)N);
#pragma omp for schedule(static)
        for (int32_t b = 0; b < B; ++b) {
            const real *h = ent + (size_t)heads[b] * d, *r = rel + (size_t)rels[b] * kw;
            const real *w = relw_row(relw, rels[b], d);
            real fp = score_one(c->score, c->p_norm, d, 0, h, r, w, ent + (size_t)tails[b] * d, scratch);
            for (int32_t n = 0; n < N; ++n)
                Frow[n] = score_one(c->score, c->p_norm, d, c->bf16_operands, h, r, w,
                                    ent + (size_t)negs[n] * d, scratch);
            Lrow[b] = row_loss(c, fp, Frow, N, w_fixed ? w_fixed + (size_t)b * N : NULL, NULL, NULL);
            if (fpos_out) fpos_out[b] = fp;
            if (F_out) memcpy(F_out + (size_t)b * N, Frow, sizeof(real) * (size_t)N);
        }
        free(scratch); free(Frow);
    }
    for (int32_t b = 0; b < B; ++b) { total += (double)Lrow[b]; if (Lrow_out) Lrow_out[b] = Lrow[b]; }
    free(Lrow);
    return c->loss_scale * total + batch_regulariser(c, ent, heads, tails, negs);
}

/*
 * Forward + backward of one batch at the given tables.  Outputs (all overwritten):
 *   dh[B,d], dtpos[B,d], dr[B,kw], dw[B,d] (TransH, else may be NULL), dtneg[N,d],
 *   G[B,N] = loss_scale * dL_b/dF_bn, gpos[B] = loss_scale * dL_b/df+_b.
 * dT_n sums over b ascending; dh_b etc. sum the positive first, then n ascending.
 */
double kgeo_batch_grads(const kgeo_config *c, const real *ent, const real *rel, const real *relw,
                        const int32_t *heads, const int32_t *rels, const int32_t *tails,
                        const int32_t *negs,
                        real *dh, real *dtpos, real *dr, real *dw, real *dtneg,
                        real *G, real *gpos) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    const int kw = rel_width(c->score, d);
    const real ls = (real)c->loss_scale;
    real *Lrow = (real *)malloc(sizeof(real) * (size_t)B);
    memset(dh, 0, sizeof(real) * (size_t)B * d);
    memset(dtpos, 0, sizeof(real) * (size_t)B * d);
    memset(dr, 0, sizeof(real) * (size_t)B * kw);
    if (dw) memset(dw, 0, sizeof(real) * (size_t)B * d);
    memset(dtneg, 0, sizeof(real) * (size_t)N * d);
#pragma omp parallel
    {
        real *scratch = (real *)malloc(sizeof(real) * 6 * (size_t)d);
        real *Frow = (real *)malloc(sizeof(real) * (size_t)N);
#pragma omp for schedule(static)
        for (int32_t b = 0; b < B; ++b) {
            const real *h = ent + (size_t)heads[b] * d, *r = rel + (size_t)rels[b] * kw;
            const real *w = relw_row(relw, rels[b], d);
            const real *tp = ent + (size_t)tails[b] * d;
            real fp = score_one(c->score, c->p_norm, d, 0, h, r, w, tp, scratch);
            for (int32_t n = 0; n < N; ++n)
                Frow[n] = score_one(c->score, c->p_norm, d, c->bf16_operands, h, r, w,
                                    ent + (size_t)negs[n] * d, scratch);
            real gp;
            real *Gb = G + (size_t)b * N;
            Lrow[b] = row_loss(c, fp, Frow, N, NULL, &gp, Gb);
            gp *= ls; gpos[b] = gp;
            for (int32_t n = 0; n < N; ++n) Gb[n] *= ls;
            real *dhb = dh + (size_t)b * d, *drb = dr + (size_t)b * kw;
            real *dwb = dw ? dw + (size_t)b * d : NULL;
            score_grad_one(c->score, c->p_norm, d, gp, h, r, w, tp, dhb, drb, dwb,
                           dtpos + (size_t)b * d, scratch);
            for (int32_t n = 0; n < N; ++n)
                score_grad_one(c->score, c->p_norm, d, Gb[n], h, r, w, ent + (size_t)negs[n] * d,
                               dhb, drb, dwb, NULL, scratch);
        }
#pragma omp for schedule(static)
        for (int32_t n = 0; n < N; ++n) {
            const real *tn = ent + (size_t)negs[n] * d;
            for (int32_t b = 0; b < B; ++b)
                score_grad_one(c->score, c->p_norm, d, G[(size_t)b * N + n],
                               ent + (size_t)heads[b] * d, rel + (size_t)rels[b] * kw,
                               relw_row(relw, rels[b], d), tn, NULL, NULL, NULL,
                               dtneg + (size_t)n * d, scratch);
        }
        free(scratch); free(Frow);
    }
    if (c->reg_lambda != 0) {   /* one term per occurrence: its gradient joins that occurrence's row */
        const real lam = (real)c->reg_lambda;
        for (int32_t b = 0; b < B; ++b) {
            l3_term_grad(c->reg_form, d, lam, ent + (size_t)heads[b] * d, dh + (size_t)b * d);
            l3_term_grad(c->reg_form, d, lam, ent + (size_t)tails[b] * d, dtpos + (size_t)b * d);
        }
        for (int32_t n = 0; n < N; ++n) l3_term_grad(c->reg_form, d, lam, ent + (size_t)negs[n] * d, dtneg + (size_t)n * d);
    }
    double total = 0;
    for (int32_t b = 0; b < B; ++b) total += (double)Lrow[b];
    free(Lrow);
    return c->loss_scale * total + batch_regulariser(c, ent, heads, tails, negs);
}

/* ------------------------------------------------------------------------- */
/* Deterministic de-duplication and sparse row update.                         */
/* ------------------------------------------------------------------------- */

/*
 * Stable sort of positions 0..n-1 by ids[pos]: perm (sorted positions), uniq (distinct
 * ids ascending), seg_off (uniq[u] owns perm[seg_off[u] .. seg_off[u+1])).  Returns U.
 */
int32_t kgeo_dedup(const int32_t *ids, int32_t n, int32_t *uniq, int32_t *seg_off, int32_t *perm) {
    /* insertion by merge: plain stable merge sort on positions */
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    for (int32_t i = 0; i < n; ++i) perm[i] = i;
    for (int32_t width = 1; width < n; width *= 2) {
        for (int32_t lo = 0; lo < n; lo += 2 * width) {
            int32_t mid = lo + width < n ? lo + width : n, hi = lo + 2 * width < n ? lo + 2 * width : n;
            int32_t a = lo, b = mid, o = lo;
            while (a < mid && b < hi) tmp[o++] = (ids[perm[b]] < ids[perm[a]]) ? perm[b++] : perm[a++];
            while (a < mid) tmp[o++] = perm[a++];
            while (b < hi) tmp[o++] = perm[b++];
        }
        memcpy(perm, tmp, sizeof(int32_t) * (size_t)n);
    }
    free(tmp);
    int32_t U = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (i == 0 || ids[perm[i]] != ids[perm[i - 1]]) { uniq[U] = ids[perm[i]]; seg_off[U] = i; ++U; }
    }
    seg_off[U] = n;
    return U;
}

/*
 * Apply one optimiser step to the rows uniq[0..U) of `table` [rows, width].
 * grad_rows[pos] points at the gradient row of source position pos; the row gradient is
 * the sum over the segment in ascending position.  state: Adam [rows, 2*width] (m | v),
 * row-wise Adagrad [rows]; unused for SGD.  `step` is the global 0-based step
 * (Adam bias correction uses step + 1 for every row, touched or not before).
 */
void kgeo_update_rows(const kgeo_config *c, double lr, uint64_t step, real *table, real *state,
                      int32_t width, const int32_t *uniq, const int32_t *seg_off, const int32_t *perm,
                      int32_t U, const real *const *grad_rows) {
    const real b1 = (real)c->beta1, b2 = (real)c->beta2, eps = (real)c->eps, lrr = (real)lr;
    real *g = (real *)malloc(sizeof(real) * (size_t)width);
    for (int32_t u = 0; u < U; ++u) {
        for (int k = 0; k < width; ++k) g[k] = 0;
        for (int32_t s = seg_off[u]; s < seg_off[u + 1]; ++s) {
            const real *gr = grad_rows[perm[s]];
            for (int k = 0; k < width; ++k) g[k] += gr[k];
        }
        real *prow = table + (size_t)uniq[u] * width;
        if (c->opt == OPT_SGD) {
            for (int k = 0; k < width; ++k) prow[k] -= lrr * g[k];
        } else if (c->opt == OPT_ADAM) {
            real *m = state + (size_t)uniq[u] * 2 * width, *v = m + width;
            real c1 = 1 - (real)pow((double)b1, (double)(step + 1));
            real c2 = 1 - (real)pow((double)b2, (double)(step + 1));
            for (int k = 0; k < width; ++k) {
                m[k] = b1 * m[k] + (1 - b1) * g[k];
                v[k] = b2 * v[k] + (1 - b2) * g[k] * g[k];
                prow[k] -= lrr * (m[k] / c1) / (R_SQRT(v[k] / c2) + eps);
            }
        } else { /* row-wise Adagrad: one accumulator per row, fed the mean square */
            real ms = 0;
            for (int k = 0; k < width; ++k) ms += g[k] * g[k];
            ms /= (real)width;
            state[uniq[u]] += ms;
            real den = R_SQRT(state[uniq[u]]) + eps;
            for (int k = 0; k < width; ++k) prow[k] -= lrr * g[k] / den;
        }
    }
    free(g);
}

/*
 * One whole training step on the given batch, in place: gradients at the pre-step tables,
 * dedup of [heads | tails | negs] and of rels, then the row updates.  relw / state
 * pointers may be NULL when unused.  Returns the batch loss.
 */
double kgeo_train_step(const kgeo_config *c, double lr, uint64_t step,
                       real *ent, real *rel, real *relw,
                       real *ent_state, real *rel_state, real *relw_state,
                       const int32_t *heads, const int32_t *rels, const int32_t *tails,
                       const int32_t *negs) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    const int kw = rel_width(c->score, d);
    real *dh = (real *)malloc(sizeof(real) * (size_t)B * d);
    real *dtp = (real *)malloc(sizeof(real) * (size_t)B * d);
    real *dr = (real *)malloc(sizeof(real) * (size_t)B * kw);
    real *dw = relw ? (real *)malloc(sizeof(real) * (size_t)B * d) : NULL;
    real *dtn = (real *)malloc(sizeof(real) * (size_t)N * d);
    real *G = (real *)malloc(sizeof(real) * (size_t)B * N);
    real *gpos = (real *)malloc(sizeof(real) * (size_t)B);
    double loss = kgeo_batch_grads(c, ent, rel, relw, heads, rels, tails, negs, dh, dtp, dr, dw, dtn, G, gpos);

    const int32_t ne = 2 * B + N;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne);
    int32_t *uniq = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne);
    int32_t *seg = (int32_t *)malloc(sizeof(int32_t) * ((size_t)ne + 1));
    int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne);
    const real **rows = (const real **)malloc(sizeof(real *) * (size_t)ne);
    for (int32_t b = 0; b < B; ++b) {
        ids[b] = heads[b]; rows[b] = dh + (size_t)b * d;
        ids[B + b] = tails[b]; rows[B + b] = dtp + (size_t)b * d;
    }
    for (int32_t n = 0; n < N; ++n) { ids[2 * B + n] = negs[n]; rows[2 * B + n] = dtn + (size_t)n * d; }
    int32_t U = kgeo_dedup(ids, ne, uniq, seg, perm);
    kgeo_update_rows(c, lr, step, ent, ent_state, d, uniq, seg, perm, U, rows);

    for (int32_t b = 0; b < B; ++b) rows[b] = dr + (size_t)b * kw;
    U = kgeo_dedup(rels, B, uniq, seg, perm);
    kgeo_update_rows(c, lr, step, rel, rel_state, kw, uniq, seg, perm, U, rows);
    if (relw) {
        for (int32_t b = 0; b < B; ++b) rows[b] = dw + (size_t)b * d;
        kgeo_update_rows(c, lr, step, relw, relw_state, d, uniq, seg, perm, U, rows);
    }
    free(dh); free(dtp); free(dr); free(dw); free(dtn); free(G); free(gpos);
    free(ids); free(uniq); free(seg); free(perm); free(rows);
    return loss;
}

/* ------------------------------------------------------------------------- */
/* Encoder (Section 3.1 "Encoder", Eq. 1): the embedding of an entity is its     */
/* trainable shallow row plus a linear projection of its fixed text features,     */
/*   e = e_S + M_H e_F  as a head,   e = e_S + M_T e_F  as a tail (positive or     */
/* negative), M_H, M_T in R^{d x |e_F|} trainable (optionally one shared matrix).  */
/* The batch functions below build the final embeddings of the batch's 2B + N      */
/* slots [heads | tails | negs] as a compact table and hand it to the functions    */
/* above, so that scores, losses and their derivatives are exactly those already   */
/* pinned; the chain rule then gives                                               */
/*   dL/de_S[id] += dL/de[slot]   and   dL/dM_X += dL/de[slot] (x) e_F[id].         */
/* bf16_projection = 1 rounds M to bf16 inside the projection (the features are     */
/* stored as bf16 values already), as the tensor-core projection does.              */
/* ------------------------------------------------------------------------- */
static void encoder_slots(const kgeo_config *c, int32_t F, const real *ent, const real *feat,
                          const real *MH, const real *MT,
                          const int32_t *heads, const int32_t *tails, const int32_t *negs, real *slots) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    for (int32_t s = 0; s < 2 * B + N; ++s) {
        const int32_t id = s < B ? heads[s] : (s < 2 * B ? tails[s - B] : negs[s - 2 * B]);
        const real *M = s < B ? MH : MT;
        const real *f = feat + (size_t)id * F;
        for (int k = 0; k < d; ++k) {
            real acc = 0;
            for (int j = 0; j < F; ++j) {
                real m = M[(size_t)k * F + j];
                acc = R_FMA(c->bf16_projection ? bf16_round(m) : m, f[j], acc);
            }
            slots[(size_t)s * d + k] = ent[(size_t)id * d + k] + acc;
        }
    }
}

static void slot_batch(int32_t B, int32_t N, int32_t *h, int32_t *t, int32_t *n) {
    for (int32_t b = 0; b < B; ++b) { h[b] = b; t[b] = B + b; }
    for (int32_t i = 0; i < N; ++i) n[i] = 2 * B + i;
}

/* Batch loss with the encoder (feat: [E, F] features, MH / MT: [d, F]). */
double kgeo_encoder_batch_loss(const kgeo_config *c, int32_t F, const real *ent, const real *feat,
                               const real *MH, const real *MT, const real *rel, const real *relw,
                               const int32_t *heads, const int32_t *rels, const int32_t *tails, const int32_t *negs) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    real *slots = (real *)malloc(sizeof(real) * (size_t)(2 * B + N) * d);
    int32_t *sh = (int32_t *)malloc(sizeof(int32_t) * (size_t)(2 * B + N)), *st = sh + B, *sn = sh + 2 * B;
    encoder_slots(c, F, ent, feat, MH, MT, heads, tails, negs, slots);
    slot_batch(B, N, sh, st, sn);
    kgeo_config cc = *c; cc.num_entities = 2 * B + N;
    double loss = kgeo_batch_loss(&cc, slots, rel, relw, sh, rels, st, sn, NULL, NULL, NULL, NULL);
    free(slots); free(sh);
    return loss;
}

/*
 * Gradients with the encoder.  Outputs: the per-slot rows dh[B,d], dtpos[B,d], dtneg[N,d] (= dL/de of the slot,
 * which is also the gradient of the slot's shallow row), dr, dw as in kgeo_batch_grads, and the dense dMH[d,F],
 * dMT[d,F] (overwritten; with MH == MT the caller adds the two).
 */
double kgeo_encoder_batch_grads(const kgeo_config *c, int32_t F, const real *ent, const real *feat,
                                const real *MH, const real *MT, const real *rel, const real *relw,
                                const int32_t *heads, const int32_t *rels, const int32_t *tails, const int32_t *negs,
                                real *dh, real *dtpos, real *dr, real *dw, real *dtneg, real *dMH, real *dMT) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    real *slots = (real *)malloc(sizeof(real) * (size_t)(2 * B + N) * d);
    int32_t *sh = (int32_t *)malloc(sizeof(int32_t) * (size_t)(2 * B + N)), *st = sh + B, *sn = sh + 2 * B;
    real *G = (real *)malloc(sizeof(real) * (size_t)B * N), *gpos = (real *)malloc(sizeof(real) * (size_t)B);
    encoder_slots(c, F, ent, feat, MH, MT, heads, tails, negs, slots);
    slot_batch(B, N, sh, st, sn);
    kgeo_config cc = *c; cc.num_entities = 2 * B + N;
    double loss = kgeo_batch_grads(&cc, slots, rel, relw, sh, rels, st, sn, dh, dtpos, dr, dw, dtneg, G, gpos);
    memset(dMH, 0, sizeof(real) * (size_t)d * F);
    memset(dMT, 0, sizeof(real) * (size_t)d * F);
    for (int32_t s = 0; s < 2 * B + N; ++s) {          /* slots in ascending order */
        const int32_t id = s < B ? heads[s] : (s < 2 * B ? tails[s - B] : negs[s - 2 * B]);
        const real *g = s < B ? dh + (size_t)s * d : (s < 2 * B ? dtpos + (size_t)(s - B) * d : dtneg + (size_t)(s - 2 * B) * d);
        real *dM = s < B ? dMH : dMT;
        const real *f = feat + (size_t)id * F;
        for (int k = 0; k < d; ++k)
            for (int j = 0; j < F; ++j) dM[(size_t)k * F + j] += g[k] * f[j];
    }
    free(slots); free(sh); free(G); free(gpos);
    return loss;
}

/* Dense optimiser step on a [rows, width] matrix (the projection matrices): every row is "touched". */
static void update_dense(const kgeo_config *c, double lr, uint64_t step, real *M, real *state, int32_t rows, int32_t width, const real *g) {
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)rows * 3 + sizeof(int32_t));
    int32_t *uniq = ids, *seg = ids + rows, *perm = ids + 2 * rows + 1;
    const real **gr = (const real **)malloc(sizeof(real *) * (size_t)rows);
    for (int32_t r = 0; r < rows; ++r) { uniq[r] = r; seg[r] = r; perm[r] = r; gr[r] = g + (size_t)r * width; }
    seg[rows] = rows;
    kgeo_update_rows(c, lr, step, M, state, width, uniq, seg, perm, rows, gr);
    free(ids); free(gr);
}

/*
 * One training step with the encoder, in place: shallow rows, relation rows (and normals) as in kgeo_train_step, the
 * projection matrices by the same optimiser rule applied densely (Adam state [d, 2F]; row-wise Adagrad one value per
 * row of M).  shared != 0: MH and MT are one matrix (pass the same pointer twice) and its gradient is dMH + dMT.
 */
double kgeo_encoder_train_step(const kgeo_config *c, int32_t F, int32_t shared, double lr, uint64_t step,
                               real *ent, const real *feat, real *MH, real *MT, real *rel, real *relw,
                               real *ent_state, real *MH_state, real *MT_state, real *rel_state, real *relw_state,
                               const int32_t *heads, const int32_t *rels, const int32_t *tails, const int32_t *negs) {
    const int32_t B = c->batch, N = c->num_neg, d = c->dim;
    const int kw = rel_width(c->score, d);
    real *dh = (real *)malloc(sizeof(real) * (size_t)B * d), *dtp = (real *)malloc(sizeof(real) * (size_t)B * d);
    real *dr = (real *)malloc(sizeof(real) * (size_t)B * kw), *dw = relw ? (real *)malloc(sizeof(real) * (size_t)B * d) : NULL;
    real *dtn = (real *)malloc(sizeof(real) * (size_t)N * d);
    real *dMH = (real *)malloc(sizeof(real) * (size_t)d * F), *dMT = (real *)malloc(sizeof(real) * (size_t)d * F);
    double loss = kgeo_encoder_batch_grads(c, F, ent, feat, MH, MT, rel, relw, heads, rels, tails, negs, dh, dtp, dr, dw, dtn, dMH, dMT);
    const int32_t ne = 2 * B + N;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne), *uniq = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne);
    int32_t *seg = (int32_t *)malloc(sizeof(int32_t) * ((size_t)ne + 1)), *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)ne);
    const real **rows = (const real **)malloc(sizeof(real *) * (size_t)ne);
    for (int32_t b = 0; b < B; ++b) { ids[b] = heads[b]; rows[b] = dh + (size_t)b * d; ids[B + b] = tails[b]; rows[B + b] = dtp + (size_t)b * d; }
    for (int32_t n = 0; n < N; ++n) { ids[2 * B + n] = negs[n]; rows[2 * B + n] = dtn + (size_t)n * d; }
    int32_t U = kgeo_dedup(ids, ne, uniq, seg, perm);
    kgeo_update_rows(c, lr, step, ent, ent_state, d, uniq, seg, perm, U, rows);
    for (int32_t b = 0; b < B; ++b) rows[b] = dr + (size_t)b * kw;
    U = kgeo_dedup(rels, B, uniq, seg, perm);
    kgeo_update_rows(c, lr, step, rel, rel_state, kw, uniq, seg, perm, U, rows);
    if (relw) {
        for (int32_t b = 0; b < B; ++b) rows[b] = dw + (size_t)b * d;
        kgeo_update_rows(c, lr, step, relw, relw_state, d, uniq, seg, perm, U, rows);
    }
    if (shared) {
        for (size_t i = 0; i < (size_t)d * F; ++i) dMH[i] += dMT[i];
        update_dense(c, lr, step, MH, MH_state, d, F, dMH);
    } else {
        update_dense(c, lr, step, MH, MH_state, d, F, dMH);
        update_dense(c, lr, step, MT, MT_state, d, F, dMT);
    }
    free(dh); free(dtp); free(dr); free(dw); free(dtn); free(dMH); free(dMT);
    free(ids); free(uniq); free(seg); free(perm); free(rows);
    return loss;
}

/* ------------------------------------------------------------------------- */
/* Full-entity inference (Section 3.1 "Inference"): every entity is a          */
/* candidate tail, order = (score descending, id ascending); MRR as in the     */
/* task description (reciprocal rank 0 beyond the cut-off).                    */
/* ------------------------------------------------------------------------- */
static int better(real fa, int64_t ia, real fb, int64_t ib) {
    return fa > fb || (fa == fb && ia < ib);
}

/*
 * For each query (qh, qr): out_ids/out_scores [nq, K] = the K best entities among
 * [ent_lo, ent_hi) (unused places: id -1, score -inf); ranks[q] = 1 + number of entities
 * in that range ordered before the true tail (whose own score uses the same arithmetic).
 */
int kgeo_score_all_topk(const kgeo_config *c, const real *ent, const real *rel, const real *relw,
                        const int32_t *qh, const int32_t *qr, int32_t nq, int32_t K,
                        const int32_t *true_tails, int64_t ent_lo, int64_t ent_hi,
                        int32_t *out_ids, real *out_scores, int64_t *ranks) {
    const int32_t d = c->dim;
    const int kw = rel_width(c->score, d);
    if (K <= 0 || ent_lo < 0 || ent_hi > c->num_entities) return ERR_BAD_ARG;
#pragma omp parallel
    {
        real *scratch = (real *)malloc(sizeof(real) * 3 * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int32_t q = 0; q < nq; ++q) {
            const real *h = ent + (size_t)qh[q] * d, *r = rel + (size_t)qr[q] * kw;
            const real *w = relw_row(relw, qr[q], d);
            int32_t *ids = out_ids + (size_t)q * K;
            real *sc = out_scores + (size_t)q * K;
            for (int32_t k = 0; k < K; ++k) { ids[k] = -1; sc[k] = -(real)INFINITY; }
            real ftrue = 0; int64_t beat = 0; int64_t tt = -1;
            if (true_tails) {
                tt = true_tails[q];
                ftrue = score_one(c->score, c->p_norm, d, c->bf16_operands, h, r, w, ent + (size_t)tt * d, scratch);
            }
            int32_t filled = 0;
            for (int64_t e = ent_lo; e < ent_hi; ++e) {
                real f = score_one(c->score, c->p_norm, d, c->bf16_operands, h, r, w, ent + (size_t)e * d, scratch);
                if (true_tails && better(f, e, ftrue, tt)) ++beat;
                if (filled == K && !better(f, e, sc[K - 1], ids[K - 1])) continue;
                int32_t pos = filled < K ? filled : K - 1;   /* insertion into the sorted list */
                while (pos > 0 && better(f, e, sc[pos - 1], ids[pos - 1])) {
                    sc[pos] = sc[pos - 1]; ids[pos] = ids[pos - 1]; --pos;
                }
                sc[pos] = f; ids[pos] = (int32_t)e;
                if (filled < K) ++filled;
            }
            if (ranks) ranks[q] = true_tails ? 1 + beat : 0;
        }
        free(scratch);
    }
    return ERR_OK;
}

/* ------------------------------------------------------------------------- */
/* Power-rank ensemble (Section 3.2 "Ensemble", Eq. 2).  lists[m][q][0..K) are  */
/* model m's top-K tails of query q in rank order (-1 = unused place).  Brute     */
/* force: every entity that occurs in one of the query's lists gets                */
/*   s(t) = sum over m ascending of  -sgn(p) k^p  if t is the k-th of list m,       */
/*                                   -[p > 0] (K + 1)^p  if t is not in list m,     */
/* and the top_n by (s descending, id ascending) are returned (entities in no list  */
/* have the lowest possible score and cannot reach the top when K >= top_n).        */
/* Always fp64.                                                                     */
/* ------------------------------------------------------------------------- */
int kgeo_ensemble_topk(const int32_t *lists, int32_t M, int32_t nq, int32_t K, double p, int32_t top_n,
                       int32_t *out_ids, double *out_scores) {
    if (M <= 0 || K <= 0 || top_n <= 0 || p == 0.0) return ERR_BAD_ARG;
    const double sgn = p > 0 ? 1.0 : -1.0;
    const double absent = p > 0 ? -pow((double)K + 1.0, p) : 0.0;
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)M * K);
    double *cs = (double *)malloc(sizeof(double) * (size_t)M * K);
    for (int32_t q = 0; q < nq; ++q) {
        int32_t nc = 0;
        for (int32_t m = 0; m < M; ++m)
            for (int32_t k = 0; k < K; ++k) {
                int32_t id = lists[((size_t)m * nq + q) * K + k];
                if (id < 0) continue;
                int seen = 0;
                for (int32_t c = 0; c < nc; ++c) if (cand[c] == id) { seen = 1; break; }
                if (!seen) cand[nc++] = id;
            }
        for (int32_t c = 0; c < nc; ++c) {
            double s = 0;
            for (int32_t m = 0; m < M; ++m) {
                int present = 0;
                for (int32_t k = 0; k < K; ++k)
                    if (lists[((size_t)m * nq + q) * K + k] == cand[c]) { s += -sgn * pow((double)(k + 1), p); present = 1; }
                if (!present) s += absent;
            }
            cs[c] = s;
        }
        for (int32_t r = 0; r < top_n; ++r) {
            int32_t best = -1;
            for (int32_t c = 0; c < nc; ++c)
                if (cand[c] >= 0 && (best < 0 || cs[c] > cs[best] || (cs[c] == cs[best] && cand[c] < cand[best]))) best = c;
            out_ids[(size_t)q * top_n + r] = best >= 0 ? cand[best] : -1;
            out_scores[(size_t)q * top_n + r] = best >= 0 ? cs[best] : -(double)INFINITY;
            if (best >= 0) cand[best] = -1;
        }
    }
    free(cand); free(cs);
    return ERR_OK;
}

/* Learning rate decayed linearly to zero over the course of training (Section 5). */
double kgeo_lr_linear_decay(double lr0, uint64_t step, uint64_t total_steps) {
    if (total_steps == 0 || step >= total_steps) return 0.0;
    return lr0 * (1.0 - (double)step / (double)total_steps);
}

/* mean over queries of (rank <= k_cut ? 1/rank : 0); k_cut = 0 means no cut-off. */
double kgeo_mrr(const int64_t *ranks, int32_t nq, int32_t k_cut) {
    double s = 0;
    for (int32_t q = 0; q < nq; ++q)
        if (k_cut <= 0 || ranks[q] <= k_cut) s += 1.0 / (double)ranks[q];
    return nq > 0 ? s / nq : 0.0;
}
