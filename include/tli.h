/*
 * tli.h -- C ABI of the Token-Level Intersection (TLI) verification library
 * for NVIDIA B200 (sm_100a).
 *
 * One call verifies K drafted tokens for each of B sequences when the drafter
 * and the target model use different vocabularies: Algorithm 4 of the paper
 * (project the drafter distribution onto the vocabulary intersection and
 * renormalise it) followed by the verification half of Algorithm 5 (rejection
 * test per draft, first rejection, residual or bonus sample).
 *
 * Conventions
 *   - Pointers marked [device] are device pointers owned by the caller; the
 *     library never frees or reallocates them.  Pointers marked [host] are
 *     read during the call only.
 *   - tli_verify() is asynchronous on the stream it is given, allocates
 *     nothing and does not synchronise.  It only launches kernels, so it may
 *     be recorded into a CUDA graph by stream capture and replayed; calls on
 *     one context must not overlap in time (they share the context's
 *     counters), so replays of such a graph are serialised by the caller.
 *     The same holds for tli_draft_sample(), tli_slem_verify() and
 *     tli_acceptance_rates(); tli_verify_host() adds only stream-ordered copies.
 *   - Functions return TLI_OK or a negative tli error code.  Errors in the
 *     data (a draft id outside the vocabulary, a NaN logit, a negative
 *     temperature) never fault: they set bits in row_status.
 */
#ifndef TLI_H
#define TLI_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tli_ctx tli_ctx; /* opaque, library-owned */

/* logit storage types */
enum { TLI_F32 = 0, TLI_BF16 = 1 };

/* return codes */
enum {
    TLI_OK = 0,
    TLI_ERR_ARG = -1,         /* null pointer, bad size, bad dtype, misaligned logits */
    TLI_ERR_BAD_MAP = -2,     /* id map entry out of range, or two drafter ids on one target id */
    TLI_ERR_CUDA = -3,        /* a CUDA runtime call failed (tli_last_cuda_error() says which) */
    TLI_ERR_WORKSPACE = -4,   /* workspace missing, misaligned or too small */
    TLI_ERR_UNSUPPORTED = -5, /* size beyond TLI_MAX_B / TLI_MAX_K / TLI_MAX_V */
    TLI_ERR_STATIC_SCRATCH = -6 /* tli_verify_static(): the batch needs more than TLI_STATIC_SCRATCH_BYTES */
};

/* row_status bits */
enum {
    TLI_ROW_DRAFT_RANGE = 1,      /* a draft id outside [0, V_d): treated as rejected */
    TLI_ROW_DRAFT_UNMAPPED = 2,   /* a draft id outside the intersection: rejected (q' = 0 there) */
    TLI_ROW_NONFINITE = 4,        /* NaN or +inf logit seen: accepted = 0, next_token = 0 */
    TLI_ROW_FALLBACK = 8,         /* empty intersection or zero residual mass: sampled from p instead */
    TLI_ROW_TIMEOUT = 16,         /* a bounded wait inside a kernel ran out: results not to be trusted.  Sticky: every
                                   * later call on the context reports it too, until tli_reset() */
    TLI_ROW_BAD_TEMPERATURE = 32  /* temperature negative or not finite: accepted = 0, next_token = 0 */
};

#define TLI_MAX_B 65535    /* sequences per call */
#define TLI_MAX_K 64       /* drafts per sequence */
#define TLI_MAX_V 1048576  /* vocabulary size (either side) */
#define TLI_MAX_SHARDS 64   /* vocabulary shards (tli_shard_create) */
#define TLI_STATIC_SCRATCH_BYTES 4194304 /* 4 MiB: scratch built into the library for tli_verify_static() */

/*
 * Create a context for one (target vocabulary, drafter vocabulary) pair on one
 * device.  Implements the "T cap D" of Algorithm 4 as data: id_map[x] is the
 * target id of drafter token x, or -1 when x is not in the target vocabulary.
 *
 *   out          [host]  receives the context
 *   device               CUDA device ordinal; made current during the call and
 *                        restored afterwards
 *   V_t, V_d             vocabulary sizes, 1 .. TLI_MAX_V
 *   id_map_host  [host]  int32[V_d]; every entry -1 or in [0, V_t); vocabularies
 *                        are sets of strings, so no two drafter ids may share a
 *                        target id (TLI_ERR_BAD_MAP otherwise).  Validated
 *                        before any CUDA call is made.
 *
 * The context owns device copies of the map, its inverse (target id -> drafter
 * id), a bit mask of mapped drafter ids, per-sequence completion counters and
 * an 8 MiB buffer for the per-row partial results of moderate batches (kept
 * "empty" between calls, so that the kernel that reads them can tell a result
 * that has been stored from one that has not without waiting for the whole
 * kernel that stores them; larger batches keep theirs in the workspace).
 * Because of the counters and that buffer a context serves one tli_verify() at
 * a time: calls on the same context must be ordered on one stream (or by events).
 */
int tli_create(tli_ctx **out, int device, int32_t V_t, int32_t V_d, const int32_t *id_map_host);

/* Free a context.  The caller makes sure no call using it is still running. */
int tli_destroy(tli_ctx *ctx);

/* Bytes of device scratch tli_verify() needs for (B, K, dtype); 0 on bad arguments. */
size_t tli_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype);

typedef struct {
    int32_t B;      /* sequences, 1 .. TLI_MAX_B */
    int32_t K;      /* drafts per sequence, 1 .. TLI_MAX_K */
    int32_t dtype;  /* TLI_F32 or TLI_BF16, for both logit tensors */

    /* [device] target logits [B, K+1, V_t]: row j is the target distribution
     * for the token at draft position j, row K the bonus position
     * (Algorithm 5's single batched target pass).  Strides in elements; the
     * vocabulary axis is contiguous.  The base pointer is aligned to the
     * element size; rows need no further alignment. */
    const void *target_logits;
    int64_t t_stride_b, t_stride_k;

    /* [device] drafter logits [B, K, V_d], the distributions the drafts were
     * sampled from.  Not read for temperature-0 sequences. */
    const void *drafter_logits;
    int64_t d_stride_b, d_stride_k;

    const int32_t *draft_ids;   /* [device] int32[B, K], drafter-vocabulary ids */
    const float *temperature;   /* [device] float[B]; softmax(z / tau) on both sides; 0 = arg-max */
    const float *uniforms;      /* [device] float[B, K+1] in [0, 1): column j < K drives the
                                 * acceptance test of draft j, column K the one extra token */

    int32_t *accepted;          /* [device] out int32[B]: accepted drafts n, 0 .. K */
    int32_t *next_token;        /* [device] out int32[B]: target-vocabulary id of the token after
                                 * the accepted drafts (residual sample if n < K, bonus sample
                                 * from row K otherwise) */
    int32_t *row_status;        /* [device] out int32[B] of TLI_ROW_* bits; may be NULL */
    float *p_draft;             /* [device] out float[B, K]: p(map[d_j]); may be NULL */
    float *q_draft;             /* [device] out float[B, K]: q'(d_j); may be NULL.  Both are 0
                                 * for temperature-0 sequences and invalid drafts */

    void *workspace;            /* [device] scratch, 256-byte aligned, >= tli_workspace_bytes();
                                 * contents need no initialisation and are garbage afterwards */
    size_t workspace_bytes;

    const int32_t *draft_lengths; /* [device] int32[B] or NULL.  Algorithm 5's lookahead given per
                                 * sequence: only the first draft_lengths[b] (0 .. K) drafts of
                                 * sequence b count; its later drafter rows and its target rows beyond
                                 * row draft_lengths[b] are not read, and when all counted drafts are
                                 * accepted the extra token is drawn from target row draft_lengths[b].
                                 * The extra token still uses uniforms[b, K].  NULL = K for all */
} tli_verify_args;

/*
 * Verify one batch (Algorithm 4, then Algorithm 5's acceptance loop, count and
 * final sample), per sequence b with tau = temperature[b]:
 *
 *   tau > 0:  p_j = softmax(target row j / tau);  q_j = softmax(drafter row j / tau);
 *             q'_j(x) = q_j(x) / sum_{map[y] >= 0} q_j(y) if map[x] >= 0, else 0;
 *             draft j is accepted iff uniforms[b,j] < min(1, p_j(map[d_j]) / q'_j(d_j));
 *             n = index of the first rejected draft, K if none;
 *             n < K:  next_token ~ max(0, p_n - q'_n) normalised (q' carried to target ids);
 *             n == K: next_token ~ p_K;
 *             both by inverse CDF in increasing target-id order with v = uniforms[b,K]:
 *             the smallest t whose cumulative weight exceeds v * total.
 *   tau == 0: a_j = lowest index attaining the maximum of target row j; draft j is
 *             accepted iff map[d_j] == a_j; next_token = a_n.
 *
 * All arithmetic on the vocabulary rows is fp32 with fp64 combination of
 * partial sums; temperature-0 rows are exact comparisons on the stored values.
 * A logit of -inf is a token of probability zero.  NaN or +inf flags the
 * sequence (TLI_ROW_NONFINITE, accepted = 0, next_token = 0) when it lies in a
 * row of one of the drafts that count (target and drafter rows 0 .. m-1, m = K
 * or draft_lengths[b]) or, when all of them are accepted, in the bonus row m;
 * in a drafter row only at an id inside the intersection: drafter logits
 * outside the intersection do not enter q' and are not examined.  In a
 * temperature-0 sequence a NaN never compares greater than anything, so it is
 * never the arg-max; which id wins in a row that holds a NaN before its largest
 * value is unspecified.
 *
 * Returns TLI_ERR_ARG / TLI_ERR_WORKSPACE / TLI_ERR_UNSUPPORTED for
 * host-detectable argument errors (nothing is launched) and TLI_ERR_CUDA if a
 * launch fails.  `cuda_stream` is a cudaStream_t (NULL = default stream); the
 * context's device must be current.
 */
int tli_verify(tli_ctx *ctx, const tli_verify_args *args, void *cuda_stream);

/*
 * tli_verify() for callers that have no way to obtain device scratch.
 * (The paper has no counterpart for this; it is a deployment convenience.)
 *
 * Some hosts of this library cannot allocate device memory at the moment they
 * need a verification: an inference server that handed its whole HBM budget to
 * the KV cache and weights at start-up, a decode loop where a cudaMalloc would
 * stall the device, a plugin that is given tensors but no allocator.  For them
 * this entry point does exactly what tli_verify() does, but ignores
 * args->workspace / args->workspace_bytes and uses a fixed
 * TLI_STATIC_SCRATCH_BYTES (4 MiB) array that is part of the library's device
 * image.  Inputs and outputs are still the caller's.  It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 * Cost and limits
 *   - every GPU on which the library is loaded holds those 4 MiB until the
 *     process exits, used or not;
 *   - a batch whose scratch need (tli_workspace_bytes()) exceeds the array is
 *     refused with TLI_ERR_STATIC_SCRATCH and nothing is launched; the five
 *     benchmark workloads need at most about 0.3 MiB;
 *   - the first call on each device looks up the array's device address (the
 *     context's device must be current, as for tli_verify()).  Make that first
 *     call outside any stream capture;
 *   - all calls on one device share the one array.  Two calls that overlap on
 *     the GPU (different streams, no ordering between them) corrupt each other;
 *     order them on one stream or with events.  The array keeps whatever the
 *     last call left in it; that is harmless, because each call writes every
 *     word of it before reading that word, so nothing needs to be cleared.
 */
int tli_verify_static(tli_ctx *ctx, const tli_verify_args *args, void *cuda_stream);

typedef struct {
    int32_t B, K, dtype;            /* as in tli_verify_args */
    const void *target_logits;      /* [host] [B, K+1, V_t], contiguous */
    const void *drafter_logits;     /* [host] [B, K, V_d], contiguous */
    const int32_t *draft_ids;       /* [host] int32[B, K] */
    const float *temperature;       /* [host] float[B] */
    const float *uniforms;          /* [host] float[B, K+1] */
    int32_t *accepted;              /* [host] out int32[B] */
    int32_t *next_token;            /* [host] out int32[B] */
    int32_t *row_status;            /* [host] out int32[B]; may be NULL */
    void *device_buffer;            /* [device] staging for the inputs, the outputs and the scratch of
                                     * tli_verify(): 256-byte aligned, >= tli_verify_host_buffer_bytes() */
    size_t device_buffer_bytes;
} tli_verify_host_args;

/* Bytes of device memory tli_verify_host() needs for (B, K, dtype); 0 on bad arguments. */
size_t tli_verify_host_buffer_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype);

/*
 * tli_verify() for inputs and outputs in host memory: copies the five inputs
 * to the caller's device buffer (cudaMemcpyAsync on the stream), runs the
 * verification there and copies accepted / next_token / row_status back, all
 * in stream order.  Allocates nothing and does not synchronise: the outputs
 * are valid once the caller has synchronised the stream.  With pageable host
 * memory the copies block the calling thread; pin the buffers to keep the call
 * asynchronous.  What it computes, and its errors, are tli_verify()'s.
 */
int tli_verify_host(tli_ctx *ctx, const tli_verify_host_args *args, void *cuda_stream);

typedef struct {
    int32_t B;      /* sequences, >= 1 */
    int32_t R;      /* rows of drafter logits per sequence, >= 1; B * R <= TLI_MAX_B */
    int32_t dtype;  /* TLI_F32 or TLI_BF16 */

    /* [device] drafter logits [B, R, V_d]; strides in elements, vocabulary axis
     * contiguous, base pointer aligned to the element size. */
    const void *drafter_logits;
    int64_t d_stride_b, d_stride_r;

    const float *temperature;   /* [device] float[B]; 0 = arg-max over the intersection */
    const float *uniforms;      /* [device] float[B, R] in [0, 1), one per row */

    int32_t *draft_ids;         /* [device] out int32[B, R]: the drawn drafter-vocabulary id,
                                 * always inside the intersection; -1 when none can be drawn */
    float *q_draft;             /* [device] out float[B, R]: q'(drawn id) (1 at temperature 0,
                                 * 0 when no id was drawn); may be NULL */
    int32_t *draft_status;      /* [device] out int32[B, R] of TLI_ROW_* bits (NONFINITE,
                                 * FALLBACK = empty intersection or no mass in it,
                                 * BAD_TEMPERATURE); may be NULL */

    void *workspace;            /* [device] scratch, 256-byte aligned, >= tli_draft_workspace_bytes() */
    size_t workspace_bytes;
} tli_draft_args;

/* Bytes of device scratch tli_draft_sample() needs for (B, R, dtype); 0 on bad arguments. */
size_t tli_draft_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t R, int32_t dtype);

/*
 * Draw the draft tokens: the drafter's side of Algorithm 4.  TLI has the
 * drafter sample from q' instead of q (Algorithm 5's drafting step run with
 * q'), so that every draft lies in the intersection of the vocabularies.  For
 * every sequence b and row r, with tau = temperature[b] and v = uniforms[b,r]:
 *
 *   tau > 0:  w(x) = exp((z[x] - m) / tau) if map[x] >= 0, else 0 (m = largest
 *             logit inside the intersection); q'(x) = w(x) / sum w, which equals
 *             Algorithm 4's q(x) / sum_{T cap D} q because the softmax
 *             denominator cancels; the id is found by inverse CDF in increasing
 *             drafter-id order: the smallest x whose cumulative weight exceeds
 *             v * total.
 *   tau == 0: the lowest id attaining the largest logit inside the intersection.
 *
 * The ids are what tli_verify() takes as draft_ids, and q_draft is the q'(d_j)
 * it recomputes.  One pass over the logits; arithmetic as in tli_verify().
 * A logit of -inf is an id of probability zero; NaN or +inf at an id inside
 * the intersection flags the row (-1, TLI_ROW_NONFINITE).  Logits outside the
 * intersection do not enter q' and are not examined.
 * Asynchronous on the stream, allocates nothing, only launches a kernel; it
 * uses the context's counters, so it must not overlap another call on the same
 * context.  Errors as for tli_verify().
 */
int tli_draft_sample(tli_ctx *ctx, const tli_draft_args *args, void *cuda_stream);

typedef struct {
    int32_t B;      /* sequences, >= 1 */
    int32_t M;      /* re-tokenised drafts per sequence (at most), 0 .. TLI_MAX_K; B * (M+1) <= TLI_MAX_B */
    int32_t dtype;  /* TLI_F32 or TLI_BF16 */

    /* [device] target logits [B, M+1, V_t]: row j is the target distribution
     * after the prompt and candidates t_1 .. t_j (Algorithm 2's single
     * batched target pass).  Strides in elements; vocabulary axis contiguous. */
    const void *target_logits;
    int64_t t_stride_b, t_stride_k;

    const int32_t *candidates;  /* [device] int32[B, M]: the drafts re-tokenised into target ids t_1 .. t_m */
    const int32_t *lengths;     /* [device] int32[B]: m_b in [0, M] (re-tokenisation gives each sequence its
                                 * own count); NULL = M for all.  Rows beyond m_b are not read */
    const float *temperature;   /* [device] float[B]; 0 = arg-max */
    const float *uniforms;      /* [device] float[B, M+1] in [0, 1): one per target row */

    int32_t *accepted;          /* [device] out int32[B]: matched candidates, 0 .. m_b */
    int32_t *next_token;        /* [device] out int32[B]: the sampled token at the first mismatch
                                 * (the bonus token t'_{m+1} when all m_b match) */
    int32_t *sampled;           /* [device] out int32[B, M+1]: every sampled token t'_j, -1 for rows
                                 * beyond m_b and for flagged sequences; may be NULL */
    int32_t *row_status;        /* [device] out int32[B] of TLI_ROW_* bits (NONFINITE, FALLBACK = a row
                                 * without mass, BAD_TEMPERATURE); may be NULL */

    void *workspace;            /* [device] scratch, 256-byte aligned, >= tli_slem_workspace_bytes() */
    size_t workspace_bytes;
} tli_slem_args;

/* Bytes of device scratch tli_slem_verify() needs for (B, M, dtype); 0 on bad arguments. */
size_t tli_slem_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t M, int32_t dtype);

/*
 * Exact-match verification, the device part of Algorithm 2 (string-level exact
 * matching): the drafts have been decoded to text and re-tokenised into target
 * ids t_1 .. t_m by the caller; this call samples a token t'_j from each of
 * the m+1 target rows (p_j = softmax(row j / tau), inverse CDF in increasing
 * target-id order with uniforms[b,j]; tau == 0: the lowest id attaining the
 * maximum), finds the first j with t'_j != t_j and reports accepted = j - 1
 * and next_token = t'_j (j = m+1, the bonus token, if every candidate
 * matched).  The id map of the context plays no part; rows have the context's
 * V_t entries.  One pass over the logits of rows 0 .. m_b; arithmetic and the
 * handling of -inf / NaN / +inf as in tli_verify().  A flagged sequence
 * reports accepted = 0, next_token = 0.  Asynchronous on the stream, allocates
 * nothing, uses the context's counters (no overlap with another call on the
 * same context).  Errors as for tli_verify().
 */
int tli_slem_verify(tli_ctx *ctx, const tli_slem_args *args, void *cuda_stream);

typedef struct {
    int32_t B;      /* sequences, >= 1 */
    int32_t K;      /* draft positions per sequence, 1 .. TLI_MAX_K; 2 * B * K <= TLI_MAX_B */
    int32_t dtype;  /* TLI_F32 or TLI_BF16, for both logit tensors */
    const void *target_logits;  /* [device] [B, >= K, V_t], as for tli_verify(); rows 0 .. K-1 are read */
    int64_t t_stride_b, t_stride_k;
    const void *drafter_logits; /* [device] [B, K, V_d] */
    int64_t d_stride_b, d_stride_k;
    const float *temperature;   /* [device] float[B] */
    float *mass;                /* [device] out float[B, K]: drafter mass on the intersection, sum_{T cap D} q */
    float *alpha_union;         /* [device] out float[B, K]: sum_{T cap D} min{p, q} */
    float *alpha_tli;           /* [device] out float[B, K]: sum_{T cap D} min{p, q / mass} */
    int32_t *position_status;   /* [device] out int32[B, K] of TLI_ROW_* bits; may be NULL */
    void *workspace;            /* [device] scratch, 256-byte aligned, >= tli_rates_workspace_bytes() */
    size_t workspace_bytes;
} tli_rates_args;

/* Bytes of device scratch tli_acceptance_rates() needs for (B, K, dtype); 0 on bad arguments. */
size_t tli_rates_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype);

/*
 * Expected acceptance rates of every draft position, the paper's table of
 * expected acceptance rates: with p = softmax(target row j / tau) and
 * q = softmax(drafter row j / tau) over all of D,
 *     mass        = sum_{x in T cap D} q(x)
 *     alpha_union = sum_{x in T cap D} min{p(map x), q(x)}          drafting from q
 *     alpha_tli   = sum_{x in T cap D} min{p(map x), q(x) / mass}   drafting from q' (Algorithm 4)
 * (alpha_union <= alpha_tli, Theorem 4.1).  tau == 0 gives the one-hot limit:
 * each value is 0 or 1.  An empty intersection gives zeros and
 * TLI_ROW_FALLBACK; NaN or +inf in a row gives zeros and TLI_ROW_NONFINITE.
 * Two passes over the drafter rows and one over the target rows plus one
 * gathered target logit per id of the intersection.  For choosing a drafter
 * and watching a deployment, not part of a decoding step.  Asynchronous,
 * allocates nothing, uses the context's counters.
 */
int tli_acceptance_rates(tli_ctx *ctx, const tli_rates_args *args, void *cuda_stream);

/*
 * Vocabulary-sharded verification: the same Algorithm 4 + Algorithm 5 step when
 * the logits come from tensor-parallel LM heads, each of G devices holding one
 * slice of every target row and one slice of every drafter row.  Algorithm 4's
 * denominator (the drafter mass on the intersection) and Algorithm 5's residual
 * normaliser are the two sums that cross shards; their partial values are
 * exchanged by the caller (one all-gather each) between four local calls, and
 * so is, for every sequence that rejected a draft, the one drafter row the
 * residual is formed from (a mapped pair may have its drafter id on one shard
 * and its target id on another).
 *
 * Partition: shard g of G holds target ids [g*Wt, min(V_t, (g+1)*Wt)) with
 * Wt = ceil(V_t / G), and drafter ids [g*Wd, ...) with Wd = ceil(V_d / G)
 * (tli_shard_info() reports them; trailing shards may hold fewer ids, or none).
 * The id map is the global one (drafter id -> target id).  draft_ids,
 * temperature and uniforms are replicated.
 *
 * One verification, on every shard, with `args` as for tli_verify() except that
 * target_logits / drafter_logits are this shard's slices ([B, K+1, >= its target
 * ids] / [B, K, >= its drafter ids], strides as given), workspace is at least
 * tli_shard_workspace_bytes(), and draft_lengths must be NULL:
 *
 *   tli_shard_stats(ctx, args, record)            record: tli_shard_record_bytes()
 *       all-gather the records            -> records_all [G][record]
 *   tli_shard_decide(ctx, args, records_all, rows)  rows: tli_shard_rows_bytes()
 *       writes accepted, row_status, p_draft, q_draft (identical on every shard),
 *       next_token of the sequences that need no sample, and this shard's slice
 *       of drafter row n of every sequence that rejected a draft
 *       all-gather the rows               -> rows_all [G][rows]
 *   tli_shard_weights(ctx, args, rows_all, mass)    mass: double[B][2]
 *       all-gather the masses             -> masses_all [G][B][2]
 *   tli_shard_select(ctx, args, rows_all, masses_all)
 *       next_token[b] = the sampled global target id on the one shard that holds
 *       it, -1 on the others: combine with an element-wise maximum over shards
 *       (sequences finished by tli_shard_decide carry the same value everywhere).
 *
 * All buffers are [device], 16-byte aligned; the gathered ones are the shards'
 * buffers in shard order.  Every call is asynchronous on the stream, allocates
 * nothing and touches local memory only; the all-gathers are the caller's (NCCL
 * or any other transport).  Results equal tli_verify()'s on the unsharded
 * tensors up to the order in which sums are formed.  A context made here serves
 * these calls only (tli_verify() refuses it).
 */
int tli_shard_create(tli_ctx **out, int device, int32_t V_t, int32_t V_d, const int32_t *id_map_host,
                     int32_t n_shards, int32_t shard);
int tli_shard_info(const tli_ctx *ctx, int32_t *t_begin, int32_t *t_count, int32_t *d_begin, int32_t *d_count,
                   int32_t *t_width, int32_t *d_width);
size_t tli_shard_workspace_bytes(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype);
size_t tli_shard_record_bytes(const tli_ctx *ctx, int32_t B, int32_t K);
size_t tli_shard_rows_bytes(const tli_ctx *ctx, int32_t B, int32_t dtype);
int tli_shard_stats(tli_ctx *ctx, const tli_verify_args *args, void *record_out, void *cuda_stream);
int tli_shard_decide(tli_ctx *ctx, const tli_verify_args *args, const void *records_all, void *rows_out, void *cuda_stream);
int tli_shard_weights(tli_ctx *ctx, const tli_verify_args *args, const void *rows_all, void *mass_out, void *cuda_stream);
int tli_shard_select(tli_ctx *ctx, const tli_verify_args *args, const void *rows_all, const void *masses_all, void *cuda_stream);

/*
 * How tli_verify() will run a batch of this shape on this context: [host]
 * plan[8] = { kernel launches per call, CTAs per sequence of the cluster
 * kernel (0: the tile kernels draw the extra token; up to 16 where the device
 * places thread-block clusters of that size, else up to 8), CTAs of the statistics
 * kernel, bytes per stage of its ring, bytes per segment, segments per target
 * row, segments per drafter row, shared memory of a cluster CTA }.
 */
int tli_verify_plan(const tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype, int32_t *plan);

/*
 * Measurement hook: the launches of one tli_verify() call of this shape with
 * kernels that do nothing -- the same grids, block sizes, shared memory, the
 * programmatic dependent launch and the cluster barrier -- so that the time a
 * call spends on getting through the stream can be told from the time it
 * spends on its work (the floor of a small batch).  Asynchronous.
 */
int tli_launch_probe(tli_ctx *ctx, int32_t B, int32_t K, int32_t dtype, void *cuda_stream);

/*
 * Measurement hook: tli_verify() with CUDA events recorded on `cuda_stream`
 * around each kernel.  Blocks until the call has finished and writes three
 * durations in milliseconds to [host] ms[3]: ms[0] the statistics pass over
 * all logits, ms[1] the per-sequence decision kernel (0 when the cluster kernel
 * decides and samples in one launch, see tli_set_tiled), ms[2] the sampling
 * pass over one row per sequence.  Creates and destroys four events per call;
 * not meant for the serving path.
 */
int tli_verify_profile(tli_ctx *ctx, const tli_verify_args *args, void *cuda_stream, float *ms);

/*
 * How tli_verify() and tli_verify_static() draw the extra token of Algorithm 5
 * (the residual or bonus sample) on this context.  enabled = 0 (default): by
 * size -- one kernel of one thread-block cluster per sequence (decision and
 * sample together) when a target row fits the shared memory of a cluster and
 * the batch is moderate, the tile kernels (decision, tile sums, inversion)
 * otherwise.  enabled = 1: always the tile kernels.  Both forms compute the
 * same weights element by element; they add them in different orders, so their
 * tokens can differ where uniforms[b,K] * total lies within rounding of a CDF
 * boundary.  For tests and measurements.
 */
int tli_set_tiled(tli_ctx *ctx, int enabled);

/*
 * Widest thread-block cluster the cluster kernel may use on this context.
 * Clusters of more than 8 CTAs are not portable: tli_create() asks the driver
 * once and allows 16 where it places them, 8 otherwise.  ctas = 8 narrows a
 * context to the portable size, ctas = 16 widens it again if the device has it
 * (TLI_ERR_UNSUPPORTED if not); other values: TLI_ERR_ARG.  Results do not
 * depend on it beyond the order of the fp64 additions across CTAs.  For tests
 * and measurements.                                                    [host]
 */
int tli_set_max_cluster(tli_ctx *ctx, int ctas);

/*
 * Self-test of the kernels' bounded waits.  Every wait inside the kernels (on a
 * shared-memory barrier that a bulk copy or another warp completes) gives up
 * after a fixed number of polls, records the fact and lets the kernel finish;
 * rows decided afterwards carry TLI_ROW_TIMEOUT.  This call runs a one-thread
 * kernel that waits, with the same code and a limit of `polls` (1 .. 2^22), on
 * a barrier nothing will ever complete, synchronises the stream and reports
 * through [host] gave_up whether the wait ended the way it must (1).  It does
 * not touch the context's sticky error word; the context stays usable.
 */
int tli_selftest_bounded_wait(tli_ctx *ctx, void *cuda_stream, unsigned polls, int *gave_up);

/*
 * Put the context's device-side state back to its initial value (stream-ordered
 * memsets): the completion tickets, the segment scheduler, the sticky time-out
 * word, and the context's 8 MiB buffer of partial results, which the kernels
 * leave "empty" after every call that ends normally.  Needed only after a call
 * reported TLI_ROW_TIMEOUT: the kernels of that call gave up in mid-flight, so
 * what they share with the next call is not back at its initial value, and every
 * later call would both start from it and carry the flag.  Must be ordered after the call that timed out and
 * before the next one, like any other call on the context.
 */
int tli_reset(tli_ctx *ctx, void *cuda_stream);

/* Vocabulary sizes and number of mapped drafter ids of a context. */
int tli_ctx_info(const tli_ctx *ctx, int32_t *V_t, int32_t *V_d, int32_t *n_mapped);

/* Static, human-readable name of a return code. */
const char *tli_status_string(int code);

/* Text of the last CUDA runtime error seen by this library on the calling thread ("" if none). */
const char *tli_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TLI_H */
