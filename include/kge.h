/*
 * kge.h -- C ABI of the B200 (sm_100a) library for the shared-negative scoring block of
 * BESS-style knowledge-graph-embedding training and inference.
 *
 * Conventions for every entry point
 * ---------------------------------
 * - Memory: the caller owns ALL device memory (tables, optimiser state, workspace, every
 *   id / output array).  The library owns only the host-side handle.  Unless a parameter
 *   is marked [host], a pointer is a DEVICE pointer.
 * - Streams: `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *   stream).  Calls enqueue work and return; only the entry points documented as
 *   synchronising wait for the stream.
 * - Errors: the return value is 0 (KGE_OK) or a negative kge_status.  Argument errors are
 *   detected on the host before anything is launched.  Problems found on the device (an
 *   id outside its table, a top-k candidate list that filled up) never trap: the kernel
 *   records a code in a sticky status word inside the workspace, substitutes row 0 for the
 *   offending id, and carries on; kge_get_status() reports and clears it.  Every wait of a
 *   kernel on an asynchronous copy is bounded; if one runs out the kernel records
 *   KGE_ERR_TIMEOUT and returns.
 * - Layouts: tables are row-major fp32 [rows, dim] with dim % 4 == 0 and 16-byte aligned
 *   bases.  Complex rows (RotatE, ComplEx) are interleaved (re0, im0, re1, im1, ...), the
 *   identification of C^(d/2) with R^d of the scoring-function table.  A RotatE relation
 *   row holds dim/2 phases.  TransH keeps translations in `rel` and hyperplane normals in
 *   `relw`, both [R, dim].  Adam state is [rows, 2*width] (first moment, then second
 *   moment); row-wise Adagrad state is [rows]; SGD has none.
 * - Determinism: every result is a pure function of the inputs; no floating-point atomics
 *   are used anywhere.
 */
#ifndef KGE_H_
#define KGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kge_handle kge_handle; /* host-side object */

/* Scoring functions: the table "Scoring functions" (Section 3.1). */
typedef enum { KGE_TRANSE = 0, KGE_TRANSH = 1, KGE_ROTATE = 2, KGE_DISTMULT = 3, KGE_COMPLEX = 4,
               KGE_ROTATE_REAL_L1 = 5   /* RotatE with p = 1 read literally: the sum of |x_k| over the d real coordinates of
                                           h o r - t (the scoring-function table identifies C^(d/2) with R^d), not the sum of
                                           complex moduli that KGE_ROTATE takes; with p = 2 the two are the same */
} kge_score_t;
/* Loss functions: Section 3.1 "Loss Functions". */
typedef enum { KGE_LOSS_LOGSIGMOID = 0, KGE_LOSS_SAMPLED_SOFTMAX = 1 } kge_loss_t;
/* The paper names no optimiser; these are the textbook rules applied to touched rows only. */
typedef enum { KGE_OPT_SGD = 0, KGE_OPT_ADAM = 1, KGE_OPT_ROWWISE_ADAGRAD = 2 } kge_opt_t;
/* Arithmetic of the B x N score block (and of full-entity scoring). */
typedef enum { KGE_PREC_FP32 = 0, KGE_PREC_BF16_TC = 1 } kge_prec_t;

typedef enum {
    KGE_OK = 0,
    KGE_ERR_BAD_ARG = -1,        /* NULL / out-of-range argument, misaligned pointer */
    KGE_ERR_DIVISIBILITY = -2,   /* B % P^2 (or B % P with head_part >= 0) or N % P != 0 */
    KGE_ERR_EMPTY_BUCKET = -3,   /* a triple bucket T_{i,j} or entity partition E_j that must be sampled is empty */
    KGE_ERR_WORKSPACE = -4,      /* workspace missing or smaller than kge_workspace_bytes() */
    KGE_ERR_UNSUPPORTED = -5,    /* combination not implemented */
    KGE_ERR_NOT_READY = -6,      /* tables not bound / graph not loaded */
    KGE_ERR_CUDA = -7,           /* a CUDA runtime call failed (see kge_last_cuda_error) */
    KGE_ERR_ID_RANGE = -8,       /* device: an entity / relation id was outside its table */
    KGE_ERR_TOPK_OVERFLOW = -9,  /* device: a candidate list overflowed and could not be recovered */
    KGE_ERR_NO_EXTENSION = -10,  /* used by the Python binding when the shared library is missing */
    KGE_ERR_TIMEOUT = -11        /* device: a bounded wait on an asynchronous copy ran out; the step's results are invalid */
} kge_status;

typedef struct {
    int64_t num_entities;   /* |E| */
    int64_t num_relations;  /* |R| */
    int32_t dim;            /* d: floats per entity row; % 4 == 0, <= 512; even for RotatE / ComplEx */
    int32_t score;          /* kge_score_t */
    int32_t p_norm;         /* 1 or 2 (distance models; RotatE L1 = sum of complex moduli) */
    int32_t loss;           /* kge_loss_t */
    int32_t opt;            /* kge_opt_t */
    int32_t prec;           /* kge_prec_t */
    int32_t batch;          /* B positives per step */
    int32_t num_neg;        /* N negatives shared by the whole batch (Eq. 4) */
    int32_t num_parts;      /* P logical entity partitions, shard size S = ceil(|E| / P) */
    int32_t head_part;      /* -1: slots spread evenly over all P*P buckets, bucket-major;
                               i >= 0: the micro-batch B_i of Eq. 3 (all heads in partition i) */
    int32_t sample_mode;    /* 0: cube-root relation law of Section 4 "Training"; 1: uniform over the bucket */
    int32_t contract;       /* TransH with fp32 arithmetic: where the backward's two contractions with per-pair coefficients
                               (sum_n c_bn t_n and sum_b c_bn w_b, c = -dL/dF . sum_k s_k w_k) run.  0: on the tensor cores, as
                               bf16 two-term splits of both operands with all four products accumulated in fp32 (2^-17 relative
                               per term), from 2^22 pairs per block and dim % 32 == 0 on, else on the CUDA cores in fp32;
                               1: on the tensor cores whenever dim % 32 == 0; 2: always on the CUDA cores.  Ignored elsewhere. */
    float gamma;            /* margin of the log-sigmoid loss */
    float adv_temp;         /* a >= 0, self-adversarial temperature (0 = uniform weights 1/N) */
    float ce_correction;    /* c of the sampled-softmax loss; the paper's value is log((|E|-1)/N) */
    float loss_scale;       /* batch loss = loss_scale * sum_b L_b */
    float lr;               /* default learning rate (kge_train_step takes one per call) */
    float beta1, beta2;     /* Adam */
    float eps;              /* Adam / Adagrad denominator epsilon */
    uint64_t seed;          /* sampler seed (Philox key); also keys kge_init_tables */
    float reg_lambda;       /* lambda_S >= 0 of the L3 regulariser (Section 3.1 "Regularisation"); 0 = off */
    int32_t reg_form;       /* 0: sum of the norms ||e||_3 as printed; 1: sum of the cubes ||e||_3^3 */
    int32_t feat_dim;       /* |e_F| of the feature-projection encoder (Eq. 1); 0 = no encoder; % 64 == 0 (the paper's is 768) */
    int32_t feat_shared;    /* 1: M_H and M_T are one matrix */
} kge_config;

/* Validate the configuration and create the handle.  Allocates nothing on the device. */
int kge_create(const kge_config* cfg /*[host]*/, kge_handle** out /*[host]*/);
void kge_destroy(kge_handle* h);

/* Bytes of device workspace needed for a graph of `num_triples` triples, inference batches
 * of up to `max_queries` queries and top-`topk` lists.  Zero for either means "not used". */
size_t kge_workspace_bytes(const kge_handle* h, int64_t num_triples, int32_t max_queries, int32_t topk);

/*
 * Attach caller-owned device memory.  ent [E, d]; rel [R, d] (RotatE [R, d/2]); relw [R, d]
 * for TransH, else NULL; *_state as described above or NULL for SGD; workspace of at
 * least kge_workspace_bytes() bytes, 256-byte aligned.  The workspace must be the one sized
 * with the same (num_triples, max_queries, topk).  Zero-fills the workspace header
 * asynchronously on `stream`.
 */
int kge_bind(kge_handle* h, float* ent, float* rel, float* relw,
             float* ent_state, float* rel_state, float* relw_state,
             void* workspace, size_t workspace_bytes,
             int64_t num_triples, int32_t max_queries, int32_t topk, void* stream);

/*
 * Feature-projection encoder (Section 3.1 "Encoder", Eq. 1; handles created with feat_dim = F > 0): the embedding of an
 * entity is its shallow row plus a linear projection of its fixed text features, e = e_S + M_H e_F as a head and
 * e = e_S + M_T e_F as a (positive or negative) tail.  feat: [E, F] bf16 features (read only); MH, MT: [d, F] fp32
 * trainable matrices (the same pointer twice when feat_shared = 1); *_state: their optimiser state (Adam [d, 2F],
 * row-wise Adagrad [d], NULL for SGD).  Call after kge_bind.  kge_train_step then projects the features of the batch's
 * 2B + N slots on tensor cores (bf16 operands, fp32 accumulation -- the (B + N) |e_F| d term of the cost model in
 * Section 4.1), adds the projections to the gathered rows, and after the backward forms dM_H = sum_b dL/de_b (x) e_F and
 * dM_T likewise (tensor cores, gradient rows rounded to bf16) and steps the matrices with the handle's optimiser, every
 * row of a matrix touched; the shallow rows' gradients are the slots' gradient rows as before.  The regulariser applies to
 * the final embeddings (Omega_T).  Full-entity scoring is not offered on handles with an encoder (KGE_ERR_UNSUPPORTED).
 */
int kge_bind_features(kge_handle* h, const uint16_t* feat, float* MH, float* MT, float* MH_state, float* MT_state, void* stream);

/*
 * Graph preprocessing (Section 4 "Partitioning"): logical partition part(e) = e div S,
 * buckets T_{i,j} = {(h,r,t): part(h) = i, part(t) = j}; the triples are put in the
 * canonical order "stable sort by (i, j, r)", with per-bucket relation offsets and the
 * running sums of the integer cube-root weights w_r = floor((n_r * 2^60)^(1/3)), n_r counted
 * inside the bucket.  h, r, t: [host] int32 arrays of length n.  The sorted copy lives in the
 * workspace.  Synchronises `stream`.  KGE_ERR_EMPTY_BUCKET if a bucket or partition the
 * sampler would need is empty; KGE_ERR_BAD_ARG if an id is out of range.
 */
int kge_graph_load(kge_handle* h, const int32_t* heads /*[host]*/, const int32_t* rels /*[host]*/,
                   const int32_t* tails /*[host]*/, int64_t n, void* stream);

/*
 * The same preprocessing for triple lists that already live in device memory (heads, rels, tails:
 * device int32 [n], read only, n < 2^31), done entirely on the device: keys counted with integer
 * atomics, the canonical order made by a stable least-significant-digit radix sort of the triple
 * indices, weights in 128-bit integer arithmetic.  The result is bit-identical to kge_graph_load on
 * the same list.  Synchronises `stream`; same error codes (KGE_ERR_UNSUPPORTED if P^2 |R| > 2^31).
 */
int kge_graph_load_device(kge_handle* h, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                          int64_t n, void* stream);

/*
 * Optional initialisation of the bound tables on the device (the paper prescribes none): entity rows
 * and relation rows N(0, std^2), RotatE phases uniform in (-pi, pi), TransH normals N(0, std^2);
 * optimiser state zero.  Element (row, 4c + j) comes from word j of Philox4x32-10 with key = seed and
 * counter (row lo, row hi, c, stream) -- stream 2 entities, 3 relations, 4 normals -- through the
 * uniform u = ((word >> 9) + 1/2) 2^-23 and, for normal entries, Box-Muller on the word pairs (0, 1)
 * and (2, 3): std sqrt(-2 ln u_a) (cos, sin)(2 pi u_b).  A table is a pure function of (seed, shape).
 * Enqueues on `stream` and returns.
 */
int kge_init_tables(kge_handle* h, float std, void* stream);

/*
 * Draw the batch of step `step` (Section 4 "Training", Eq. 3 and Eq. 4): B positives, with
 * replacement, B/P^2 from every bucket (or B/P from each T_{i,j} of head_part i), the
 * relation by p(r) ~ n_r^(1/3) and the triple uniform within (bucket, r); N negatives,
 * N/P uniform entities from each partition E_j, shared by all positives.  Random words come
 * from Philox4x32-10 with key = seed and counter = (slot, step lo, step hi, stream) where
 * stream 0 draws positives and 1 negatives; a 64-bit word x maps to [0, n) as floor(x n / 2^64).
 * Outputs: heads, rels, tails [B], negs [N] int32.
 */
int kge_sample_batch(kge_handle* h, uint64_t step, int32_t* heads, int32_t* rels, int32_t* tails,
                     int32_t* negs, void* stream);

/*
 * One training step on one batch: gather rows, per-query vectors, positive scores, the
 * B x N shared-negative score block (scoring-function table), the loss (log-sigmoid with
 * self-adversarial weights under StopGrad, or sampled softmax with correction c), the
 * backward pass, de-duplication of touched rows and the sparse row update.  All gradients
 * are taken at the pre-step tables.  If heads/rels/tails/negs are all NULL the batch of
 * `step` is sampled internally exactly as kge_sample_batch would.  `step` also drives Adam's
 * bias correction (t = step + 1).  loss_out: one float, loss_scale * sum_b L_b (may be NULL).
 * With reg_lambda > 0 the L3 regulariser of Section 3.1 "Regularisation" on the gathered entity rows,
 * lambda_S Omega_S with Omega_S = sum_b (||h_b||_3 + ||t_b||_3) + sum_n ||t'_n||_3 (one term per
 * occurrence of a row; without a feature projection Omega_T = Omega_S), is added to the loss as it
 * stands (not times loss_scale) and its gradient to the rows' gradients.
 */
int kge_train_step(kge_handle* h, uint64_t step, float lr,
                   const int32_t* heads, const int32_t* rels, const int32_t* tails, const int32_t* negs,
                   float* loss_out, void* stream);

/*
 * Pieces of the training step for an entity table sharded row-wise over several devices (Section 4 "Training": worker i
 * holds the shard E_i, processes the micro-batch B_i whose heads lie in E_i, receives the rows of its B positive tails and
 * N negatives from their owners by a balanced AllToAll -- B/D + N/D rows from every worker, Eq. 3 and Eq. 4 -- and, not
 * spelled out in the paper, returns their gradient rows the same way).  The library does not communicate; the caller
 * moves the rows between devices between these calls (paper_2211_12281_b200/sharded.py does, with torch.distributed).
 *
 *   kge_gather_rows      rows_out [n, d] = the shard's rows of the n whole-table ids `ids` (all must lie in
 *                        [ent_base, ent_base + num_entities), else KGE_ERR_ID_RANGE is recorded): what an owner sends.
 *   kge_train_gradients  forward and backward of one batch exactly as kge_train_step, but nothing is de-duplicated or
 *                        updated: the gradient rows of the slots [heads | tails | negs] ([2B+N, d]), of the relations
 *                        ([B, k]) and of the TransH normals ([B, d]) stay in the workspace, where kge_gradient_rows
 *                        points.  The ids index the bound table (a worker binds its shard extended by B + N rows that
 *                        hold the received tails and negatives, and renumbers the batch accordingly).
 *   kge_apply_gradients  table (0 entities, 1 relations, 2 TransH normals) receives n (row id, gradient row) pairs:
 *                        stable sort by id, one optimiser step per distinct row with its gradients added in ascending
 *                        list position -- the step's own de-duplication and update on a list of the caller's.  scratch:
 *                        device memory of kge_apply_scratch_bytes(h, table, n) bytes, 256-byte aligned.
 * All three enqueue on `stream` and return.
 */
int kge_gather_rows(kge_handle* h, const int32_t* ids, int32_t n, int64_t ent_base, float* rows_out, void* stream);
int kge_train_gradients(kge_handle* h, uint64_t step, const int32_t* heads, const int32_t* rels, const int32_t* tails,
                        const int32_t* negs, float* loss_out, void* stream);
int kge_gradient_rows(kge_handle* h, float** grad_ent /*[host]*/, float** grad_rel /*[host]*/, float** grad_relw /*[host]*/);
size_t kge_apply_scratch_bytes(const kge_handle* h, int32_t table, int32_t n);
int kge_apply_gradients(kge_handle* h, int32_t table, const int32_t* ids, const float* grads, int32_t n, uint64_t step, float lr,
                        void* scratch, size_t scratch_bytes, void* stream);

/*
 * The same step for callers that keep the batch on the host: ids are [host] arrays (pinned
 * memory makes the copies asynchronous), copied in on `stream` (as one copy when the four
 * lists lie back to back in the order heads, rels, tails, negs); the loss is copied back to
 * *loss_out [host] and the stream is synchronised before returning.
 */
int kge_train_step_host(kge_handle* h, uint64_t step, float lr,
                        const int32_t* heads, const int32_t* rels, const int32_t* tails, const int32_t* negs,
                        float* loss_out /*[host]*/, void* stream);

/*
 * Full-entity inference (Section 3.1 "Inference"): every query (h, r, ?) is scored against
 * all |E| entities; out_ids / out_scores [nq, k] receive the k best tails ordered by
 * (score descending, entity id ascending) -- unused places (k > |E|) hold id -1 and -inf.
 * If true_tails is given, out_ranks[q] (int32) = 1 + number of entities ordered before the
 * true tail under the same order; neither the head nor the true tail is filtered.  nq must
 * not exceed the max_queries the workspace was sized for, k not its topk.  nq = 0 is a no-op that
 * returns KGE_OK (the array arguments may then be NULL).
 * Synchronises `stream` (candidate-list occupancy is checked between entity chunks).
 */
int kge_score_all_topk(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int32_t k,
                       const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                       void* stream);

/*
 * kge_score_all_topk for callers that keep queries and results on the host: q_heads, q_rels,
 * true_tails (or NULL) are [host] int32 [nq]; out_ids / out_scores [host] [nq, k]; out_ranks [host]
 * [nq] or NULL (pinned memory makes the copies asynchronous).  The queries are copied in and the
 * results copied back on `stream` through staging arrays inside the workspace; synchronises.
 */
int kge_score_all_topk_host(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int32_t k,
                            const int32_t* true_tails, int32_t* out_ids, float* out_scores, int32_t* out_ranks,
                            void* stream);

/*
 * Full-entity inference with the entity table sharded row-wise over several devices (Section 4 "Inference": the heads of
 * the queries are shared between the workers, every worker scores all queries against its own shard and returns its
 * top-K, and a final top-K over the D K gathered candidates selects the predictions).  The handle is bound to ONE shard:
 * its num_entities rows are the entities [ent_base, ent_base + num_entities) of the whole table; relation tables are whole
 * on every device.  Entity ids in q_heads, true_tails and in the outputs are ids of the whole table.  The library does
 * not communicate: between these calls the caller sums or gathers the small per-query arrays over the devices.
 *
 *   kge_shard_query_vectors  qvec_out [nq, d]: the query vector of every query whose head lies in this shard, zeros for
 *                            the others.  Summed over the shards (each head lies in exactly one) this is every query's
 *                            vector, bit for bit as a single device builds it.
 *   kge_shard_true_scores    ftrue_out [nq]: the score of the true tail, from the summed query vectors, for the true
 *                            tails that lie in this shard; zeros for the others.  Sum over the shards.
 *   kge_shard_score_topk     the summed qvec (and ftrue, true_tails, or all three NULL) against this shard: out_ids /
 *                            out_scores [nq, k] its k best tails as in kge_score_all_topk, out_beat [nq] the number of
 *                            its entities ordered before the true tail.  Synchronises `stream`.
 *   kge_merge_topk           cand_ids / cand_scores [nq, per_query] (the shards' lists side by side, per_query <= 2048,
 *                            places holding id -1 ignored) -> out_ids / out_scores [nq, k], the k best under (score
 *                            descending, id ascending).  The rank of the true tail is 1 + the sum of the shards' out_beat.
 * nq must not exceed the max_queries the workspace was sized for, k not its topk.
 */
int kge_shard_query_vectors(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, int32_t nq, int64_t ent_base,
                            float* qvec_out, void* stream);
int kge_shard_true_scores(kge_handle* h, const float* qvec, const int32_t* q_rels, const int32_t* true_tails, int32_t nq,
                          int64_t ent_base, float* ftrue_out, void* stream);
int kge_shard_score_topk(kge_handle* h, const float* qvec, const int32_t* q_rels, int32_t nq, int32_t k, const float* ftrue,
                         const int32_t* true_tails, int64_t ent_base, int32_t* out_ids, float* out_scores, int32_t* out_beat,
                         void* stream);
int kge_merge_topk(const int32_t* cand_ids, const float* cand_scores, int32_t nq, int32_t per_query, int32_t k,
                   int32_t* out_ids, float* out_scores, void* stream);

/*
 * Tensor-core inference (KGE_PREC_BF16_TC, DistMult / ComplEx) scores against a bf16 copy of the
 * entity table kept in the workspace.  The copy is made by the first kge_score_all_topk / kge_eval_mrr
 * after kge_bind and again after every kge_train_step or kge_init_tables on this handle; a caller that
 * changes the entity table by any other means must call this before the next inference call, or it will
 * score against the old rows.  Enqueues the copy on `stream` (46.6 GB read, 23.3 GB written at 91 M x 128).
 * A no-op returning KGE_OK for handles without a tensor-core inference workspace.
 */
int kge_refresh_inference_table(kge_handle* h, void* stream);

/*
 * (No counterpart in the paper: an addition for callers that cannot allocate.)
 * kge_score_all_topk for programs that must not call cudaMalloc -- an inference service whose
 * whole GPU memory is already handed to another allocator, a plugin that runs under a host
 * which forbids allocation after start-up, a loop that cannot afford the device-wide
 * synchronisation an allocation may imply.  It takes no handle and no workspace: the tables,
 * the queries and the outputs are the caller's device arrays as in kge_score_all_topk, and
 * every intermediate lives in one fixed array of 804,608 bytes that is part of the library
 * image, so each GPU that loads the library holds it until the process exits.  Only the
 * fields num_entities, num_relations, dim, score and p_norm of `cfg` [host] are read.
 * Limits of the fixed array: nq <= 64, k <= 32, dim <= 512; anything larger is refused with
 * KGE_ERR_WORKSPACE before any launch.  No device or host memory is allocated or freed.
 * The first call on a device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.  All calls share the one
 * array: it keeps the previous call's contents (this entry point clears what must start at
 * zero), and two calls that overlap on the same GPU -- from different streams or threads --
 * race on it, so serialise them.  Synchronises `stream`; returns 0, an argument error,
 * KGE_ERR_CUDA, or the code recorded on the device (KGE_ERR_ID_RANGE, KGE_ERR_TIMEOUT).
 */
int kge_score_all_topk_static(const kge_config* cfg /*[host]*/, const float* ent, const float* rel,
                              const float* relw, const int32_t* q_heads, const int32_t* q_rels, int32_t nq,
                              int32_t k, const int32_t* true_tails, int32_t* out_ids, float* out_scores,
                              int32_t* out_ranks, void* stream);

/*
 * Mean reciprocal rank of the true tails (task metric of Section 2): mean over queries of
 * 1/rank if rank <= k_cutoff else 0; k_cutoff = 10 is the paper's metric, 0 = no cut-off.
 * mrr_out: [host] double.  Synchronises `stream`.
 */
int kge_eval_mrr(kge_handle* h, const int32_t* q_heads, const int32_t* q_rels, const int32_t* true_tails,
                 int32_t nq, int32_t k_cutoff, double* mrr_out /*[host]*/, void* stream);

/*
 * The same mean over ranks the caller already has (the out_ranks of kge_score_all_topk, [nq] int32 on
 * the device), so that a caller who needs the lists and the metric scores the table once.  The sum is
 * taken in fp64 on the device in a fixed order.  mrr_out: [host] double.  Synchronises `stream`.
 */
int kge_mrr_from_ranks(kge_handle* h, const int32_t* ranks, int32_t nq, int32_t k_cutoff,
                       double* mrr_out /*[host]*/, void* stream);

/* Learning rate of step `step` when lr0 is decayed linearly to zero over total_steps steps (the
 * recipe of Section 5): lr0 (1 - step / total_steps), 0 from total_steps on.  Pure host arithmetic;
 * pass the result to kge_train_step. */
float kge_lr_linear_decay(float lr0, uint64_t step, uint64_t total_steps);

/*
 * Power-rank ensemble (Section 3.2 "Ensemble", Eq. 2).  lists: device int32 [num_models, nq, k_list],
 * lists[m][q] = the top-k_list tails of model m for query q in rank order (the out_ids of
 * kge_score_all_topk; places holding -1 are skipped).  Every entity of a query's lists gets
 * s(t) = sum over the models, in ascending model order, of table[k - 1] if t is the k-th entry of the
 * model's list and table[k_list] if it is in none of its places; out_ids [nq, top_n] receives the
 * top_n entities by (s descending, entity id ascending), out_scores [nq, top_n] (device fp64, may be
 * NULL) their s; places beyond the number of distinct entities hold -1 and -inf.  The sums are fp64
 * additions of the table's entries in that fixed order.  At most 16,384 list entries per query
 * (num_models * k_list; else KGE_ERR_WORKSPACE).  Enqueues on `stream` and returns.
 *
 * kge_ensemble_rank_scores fills the table [host, k_list + 1 doubles] for a power p != 0 as Eq. 2
 * defines it: table[k - 1] = -sgn(p) k^p for k = 1 .. k_list, table[k_list] = -(k_list + 1)^p if
 * p > 0, else 0 (the paper settles on p = -0.5).  Copy it to the device for kge_ensemble_topk.
 */
int kge_ensemble_rank_scores(double power, int32_t k_list, double* table /*[host]*/);
int kge_ensemble_topk(const int32_t* lists, int32_t num_models, int32_t nq, int32_t k_list, const double* table,
                      int32_t top_n, int32_t* out_ids, double* out_scores, void* stream);

/* Synchronise `stream`, return the sticky device status word (0 or a negative code), clear it. */
int kge_get_status(kge_handle* h, void* stream);

/* Kernels launched by this handle since creation (the library's own launches only). */
int64_t kge_launch_count(const kge_handle* h);

/*
 * Per-stage device timing for the benchmark's roofline report (not part of the method).
 * While enabled, kge_train_step brackets each of its launches with CUDA events on `stream`
 * and synchronises the stream at the end of the step to accumulate the elapsed times.
 * kge_profile_read copies the totals: ms[KGE_NUM_STAGES] and launches[KGE_NUM_STAGES]
 * ([host] arrays), stages in the order of kge_stage_t; reset != 0 clears them.
 */
typedef enum {
    KGE_STAGE_SAMPLE = 0, KGE_STAGE_BUILD, KGE_STAGE_BLOCK, KGE_STAGE_LOSS,
    KGE_STAGE_TH_U,          /* TransH with tensor-core contractions: u = w.t (operand splits + contraction) */
    KGE_STAGE_ACCUM_Q, KGE_STAGE_ACCUM_T, KGE_STAGE_CHAIN, KGE_STAGE_RANK, KGE_STAGE_SEGMENT,
    KGE_STAGE_UPDATE,
    KGE_STAGE_TH_CONTRACT,   /* the same: sum_n c_bn t_n and sum_b c_bn w_b (operand splits + both contractions) */
    KGE_NUM_STAGES
} kge_stage_t;
int kge_profile(kge_handle* h, int enable);
int kge_profile_read(kge_handle* h, double* ms /*[host]*/, int64_t* launches /*[host]*/, int reset);

/*
 * Measurement helper for the benchmark's roofline (not part of the method): the rate, in lane
 * instructions per second over the whole GPU, at which the CUDA cores retire one of the instruction
 * mixes the CUDA-core kernels consist of, from a register-resident loop of `iters` rounds:
 * mix 0 fused multiply-add; mix 1 subtract + add of the absolute value (2 per element);
 * mix 2 compare + predicated add (2 per element); mix 3 special-function exponential (counted
 * alone; its accumulating add rides along).  per_second: [host].  Allocates 256 bytes of device
 * memory for the duration of the call and synchronises.
 */
int kge_measure_alu(int32_t mix, int32_t iters, double* per_second /*[host]*/, void* stream);

const char* kge_error_string(int code);
const char* kge_last_cuda_error(const kge_handle* h);

/*
 * Parity taps (never on a timed path): copy an intermediate of the most recent
 * kge_train_step to host memory.  Synchronises `stream`.  `bytes` must match exactly;
 * kge_debug_bytes returns the size (0 if the tap does not exist for this configuration).
 */
typedef enum {
    KGE_TAP_Q = 0,         /* [B, d] per-query vectors */
    KGE_TAP_FPOS = 1,      /* [B] positive scores */
    KGE_TAP_G = 2,         /* [B, N] dL/dF (for p = 2 distance models: dL/dF divided by the distance) */
    KGE_TAP_GRAD_ENT = 3,  /* [2B+N, d] gradient rows of [heads | tails | negs] */
    KGE_TAP_GRAD_REL = 4,  /* [B, k] relation gradient rows */
    KGE_TAP_GRAD_RELW = 5, /* [B, d] TransH normal gradient rows */
    KGE_TAP_ENT_UNIQ = 6,  /* [U] int32 distinct touched entity ids, ascending */
    KGE_TAP_ENT_SEG = 7,   /* [U+1] int32 segment offsets into the permutation */
    KGE_TAP_ENT_PERM = 8,  /* [2B+N] int32 source positions, stably sorted by id */
    KGE_TAP_REL_UNIQ = 9, KGE_TAP_REL_SEG = 10, KGE_TAP_REL_PERM = 11,
    KGE_TAP_LROW = 12,     /* [B] per-positive loss */
    KGE_TAP_BATCH = 13,    /* [3B+N] int32 heads | rels | tails | negs used by the step */
    KGE_TAP_GRAPH_H = 14, KGE_TAP_GRAPH_R = 15, KGE_TAP_GRAPH_T = 16,   /* [T] int32 triples in canonical order */
    KGE_TAP_GRAPH_OFF = 17,   /* [P*P*(R+1)] int64 first sorted index of relation r in bucket (i, j) */
    KGE_TAP_GRAPH_WCUM = 18   /* [P*P*(R+1)] uint64 running sums of the cube-root weights per bucket */
} kge_tap_t;
size_t kge_debug_bytes(kge_handle* h, int tap, void* stream);
int kge_debug_export(kge_handle* h, int tap, void* dst /*[host]*/, size_t bytes, void* stream);

/*
 * Parity tap of the B x N score block F_bn = f(q_b, t_n) (scoring-function table): while scores_out
 * (a caller-owned device array of B * N floats, 16-byte aligned) is set, every kge_train_step also
 * writes the block there, row-major [B, N] -- a device copy before the loss overwrites the block on
 * the fp32 path, one extra contraction on the tensor-core path (which never stores the block).
 * NULL switches the tap off.  Never on a timed path.
 */
int kge_debug_capture_scores(kge_handle* h, float* scores_out);

/*
 * Every wait of a kernel on an asynchronous copy or a barrier is a bounded loop of `tries`
 * attempts (default 2^20, seconds in all; 0 restores the default).  A test shortens it here;
 * kge_debug_wait_probe then launches one thread block that waits on a barrier nothing arrives at:
 * the wait runs out after `tries` attempts, the kernel records KGE_ERR_TIMEOUT in the status word
 * and returns -- the give-up path every kernel of the library shares -- and the context stays usable.
 */
/* Parity tap of the table generator: the raw Philox words of kge_init_tables for a [rows, width]
 * table of stream `stream_id`, as bit patterns in out (device, rows * width words). */
int kge_debug_init_words(kge_handle* h, float* out, int64_t rows, int32_t width, uint32_t stream_id, void* stream);

int kge_debug_set_wait_limit(kge_handle* h, int32_t tries);
int kge_debug_wait_probe(kge_handle* h, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KGE_H_ */
