/*
 * aasd.h - C ABI of the B200 draft-and-verify path of Alignment-Augmented Speculative
 * Decoding (AASD).
 *
 * The library covers what surrounds the target model in one decoding step of the method
 * (Algorithm 1): alignment sampling over the prefill distributions (Sec. 2.3, Sec. 3.2,
 * Fig. 2), context-aware drafting by longest-suffix lookup (Sec. 3.1), conditional
 * verification with the entropy-adaptive threshold (Sec. 3.3, Eq. 3-6) including the
 * prefix rule (Sec. 2.1), and the choice of the longest passing candidate.  The model's
 * logits are an input.
 *
 * Conventions
 *  - Every tensor pointer is a DEVICE pointer owned by the caller unless a comment says
 *    HOST.  The library keeps no pointer after the work it enqueued has run.  Output
 *    pointers inside the *_out structs may be NULL to skip that output.
 *  - Calls enqueue work on the context's stream and return without synchronising, except
 *    aasd_poll_status / aasd_get_counters, which synchronise that stream.
 *  - The return value is an aasd_status.  Errors that the host can see (NULL required
 *    pointer, bad size, unsupported mode, workspace too small) are returned before
 *    anything is launched.  Anomalies seen on the device (token id outside the
 *    vocabulary, NaN or +inf logit, history overflow) set bits in a device status word
 *    that aasd_poll_status returns and clears; the kernels never trap.
 *  - Logits are row-major [rows x vocab] with a row stride given in elements; dtype is
 *    AASD_F32 or AASD_BF16.  Rows are streamed at close to memory speed whatever their
 *    alignment (a bf16 vocabulary of 50257 with stride = vocab is as fast as a padded one:
 *    every row is copied from its first 16-byte boundary on).  Two exceptions take a much
 *    slower path with identical results: rows shorter than 256 bytes, and calls that draw
 *    keyed samples (AASD_ALIGN_GUMBEL, AASD_VERIFY_STRICT_SAMPLED) from rows that do not all
 *    start on 16-byte boundaries - pad the row stride for those.
 *  - Token ids are int32, AASD_NONE (-1) means "no token".  Offsets arrays are CSR.
 *  - Scratch memory comes from the caller: a workspace of aasd_workspace_bytes() bytes
 *    that was registered once with aasd_workspace_init().  A workspace must not be shared
 *    by calls that may overlap on the device.
 *  - There is no CPU fallback: aasd_create fails with AASD_ERR_NOT_SM100 on a device
 *    whose compute capability is not 10.x.
 */
#ifndef AASD_H
#define AASD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AASD_NONE (-1)
#define AASD_MAX_EXTRA 4   /* upper bound of k_extra */
#define AASD_MAX_NGRAM 16  /* upper bound of the key length n */

typedef enum aasd_status {
    AASD_OK = 0,
    AASD_ERR_INVALID_ARG = 1,
    AASD_ERR_BAD_SHAPE = 2,
    AASD_ERR_BAD_DTYPE = 3,
    AASD_ERR_WORKSPACE_TOO_SMALL = 4,
    AASD_ERR_CUDA = 5,
    AASD_ERR_NOT_SM100 = 6,
    AASD_ERR_UNSUPPORTED = 7
} aasd_status;

typedef enum aasd_dtype { AASD_F32 = 0, AASD_BF16 = 1 } aasd_dtype;

/* aasd_align_params.hints / aasd_verify_params.hints: performance hints, never needed for
 * correct results. */
#define AASD_HINT_FINITE 1u /* the logits are expected to hold no -inf (no masked tokens), as a
                               language-model head produces them: the streaming pass then skips
                               the step that makes masked tokens harmless.  A row that holds -inf
                               all the same is still evaluated correctly, by a much slower second
                               pass over that row (counted in redo_rows). */

/* How the extra tokens of a misaligned position are chosen. */
typedef enum aasd_align_mode {
    AASD_ALIGN_TOPK = 0,   /* the tokens ranked above the prompt token (Fig. 2) */
    AASD_ALIGN_GUMBEL = 1  /* k_extra keyed Gumbel-max draws from the distribution */
} aasd_align_mode;

typedef enum aasd_verify_mode {
    AASD_VERIFY_CONDITIONAL = 0,   /* Eq. 4-6 for eligible tokens, strict for the others */
    AASD_VERIFY_STRICT_GREEDY = 1, /* accept iff draft == argmax (Sec. 2.1) */
    AASD_VERIFY_STRICT_SAMPLED = 2,/* accept iff draft == the row's keyed sample (Eq. 1) */
    AASD_VERIFY_TOP_K = 3          /* eligible tokens pass iff they are among the row's top_k tokens
                                      (the alternative of Sec. 3.3, ablated with k = 5 in Sec. 4.4);
                                      the others strict as in CONDITIONAL */
} aasd_verify_mode;

/* Bits of the device status word. */
#define AASD_STATUS_BAD_ROW 1u        /* a logits row held NaN/+inf or only -inf */
#define AASD_STATUS_ID_RANGE 2u       /* a token id outside [0, vocab) was ignored */
#define AASD_STATUS_HIST_OVERFLOW 4u  /* aasd_append dropped tokens: history full */
#define AASD_STATUS_BAD_OFFSETS 8u    /* a CSR array was not monotone / inconsistent */
#define AASD_STATUS_TIMEOUT 16u       /* a bounded wait inside a kernel ran out: the results of
                                         that call are invalid and the workspace must be
                                         registered again before its next use */
#define AASD_STATUS_INTERNAL 32u      /* checked builds only (compiled with AASD_BOUNDS_CHECK): an
                                         index computed inside a kernel fell outside its array;
                                         the access was skipped */

/* Bits of a draft token's flag byte (Sec. 3.3, last paragraph). */
#define AASD_FLAG_CONDITIONAL 1u /* from the input context or alignment sampling */
#define AASD_FLAG_EXTRA 2u       /* an alignment-sampled alternative */

/* aasd_draft_params.flags */
#define AASD_DRAFT_MATCH_ALIGN 1u /* the last key token may also match an extra */

typedef struct aasd_ctx aasd_ctx;

typedef struct aasd_counters {
    uint64_t rows;            /* logits rows processed */
    uint64_t bad_rows;        /* rows flagged AASD_STATUS_BAD_ROW */
    uint64_t redo_rows;       /* rows that needed the second, max-referenced pass */
    uint64_t near_threshold;  /* conditional decisions with |p - (alpha*H+beta)| <= 1e-6 */
    uint64_t accepted;        /* accepted draft rows (before the prefix rule) */
    uint64_t sampler_recheck; /* sampled rows whose leading groups were re-scored in fp64 */
    uint64_t sampler_exact;   /* sampled rows that took the exhaustive fp64 path */
    uint64_t reserved;
} aasd_counters;

/* ---- context ------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` whose work goes to `stream` (a cudaStream_t,
 * NULL = the legacy default stream).  Allocates a small device block for the status word
 * and counters.  AASD_ERR_NOT_SM100 unless the device is compute capability 10.x. */
int aasd_create(aasd_ctx** out, int device, void* stream);
int aasd_destroy(aasd_ctx* ctx);
int aasd_set_stream(aasd_ctx* ctx, void* stream);
/* Static string for a status code. */
const char* aasd_status_str(int status);
/* Synchronises the stream, returns the device status bits in *bits and clears them. */
int aasd_poll_status(aasd_ctx* ctx, uint32_t* bits);
/* Synchronises the stream and copies the running counters to *out (HOST). */
int aasd_get_counters(aasd_ctx* ctx, aasd_counters* out);
int aasd_reset_counters(aasd_ctx* ctx);
/* Number of kernels the context has launched so far (host-side count). */
uint64_t aasd_launch_count(const aasd_ctx* ctx);

/* Bytes of scratch needed by aasd_align_sample / aasd_verify / aasd_step for at most
 * max_rows logits rows and max_cands candidates per call. */
int aasd_workspace_bytes(int64_t max_rows, int64_t max_cands, size_t* bytes);
/* Registers a 256-byte aligned device buffer of at least aasd_workspace_bytes(max_rows,
 * max_cands) bytes with the context and clears it (asynchronous).  Required once before
 * the buffer's first use; the context remembers its layout by address. */
int aasd_workspace_init(aasd_ctx* ctx, void* workspace, size_t bytes, int64_t max_rows,
                        int64_t max_cands);
/* Forgets a registered workspace (the caller frees the memory). */
int aasd_workspace_release(aasd_ctx* ctx, void* workspace);

/* ---- alignment sampling (Sec. 2.3, Sec. 3.2, Fig. 2) ----------------------------- */

typedef struct aasd_align_params {
    int32_t vocab;
    int32_t dtype;          /* aasd_dtype of prefill_logits */
    int64_t row_stride;     /* elements between consecutive rows, >= vocab */
    float inv_temperature;  /* logits are multiplied by this before the softmax; > 0 */
    int32_t k_extra;        /* at most this many extras per position (paper: 2), 0..4 */
    int32_t mode;           /* aasd_align_mode */
    uint32_t stream_tag;    /* distinguishes random streams of calls sharing a seed */
    uint64_t seed;          /* key of the counter-based generator (GUMBEL mode) */
    uint32_t hints;         /* AASD_HINT_* */
} aasd_align_params;

typedef struct aasd_align_out {
    int32_t* align_ids;  /* [n_rows x k_extra] extras of the position after row t, NONE padded */
    float* align_p;      /* [n_rows x k_extra] their probabilities, 0 padded */
    int32_t* n_extra;    /* [n_rows] number of extras */
    float* p_next;       /* [n_rows] probability of the prompt's own next token (0 if none) */
    int32_t* top1;       /* [n_rows] greedy token of the row (ties: lowest id) */
    float* entropy;      /* [n_rows] entropy in nats */
    float* pmax;         /* [n_rows] largest probability */
    uint8_t* aligned;    /* [n_rows] 1 iff the next prompt token equals top1 (Sec. 2.3) */
} aasd_align_out;

/* Row t of sequence b (seq_offsets[b] <= t < seq_offsets[b+1], global row index) holds the
 * distribution of the token after prompt_ids[t]; its "next token" is prompt_ids[t+1], or
 * NONE on the last row of a sequence.  TOPK mode: the extras are those of the row's
 * k_extra best tokens (logit descending, ties by lower id) that rank above the next token;
 * all k_extra of them when there is no next token.  GUMBEL mode: aligned rows get none,
 * other rows k_extra keyed draws, keeping distinct tokens different from the next token.
 * n_rows must equal seq_offsets[n_seqs].  A bad row gets NONE/0 everywhere. */
int aasd_align_sample(aasd_ctx* ctx, const void* prefill_logits, const int32_t* prompt_ids,
                      const int32_t* seq_offsets, int32_t n_seqs, int64_t n_rows,
                      const aasd_align_params* params, void* workspace, size_t workspace_bytes,
                      const aasd_align_out* out);

/* ---- drafting (Sec. 3.1, Algorithm 1) --------------------------------------------- */

typedef struct aasd_draft_params {
    int32_t n_seqs;
    int32_t n;          /* longest key (suffix) length, 1..AASD_MAX_NGRAM (paper: 6) */
    int32_t draft_len;  /* tokens per candidate */
    int32_t max_cands;  /* candidates per sequence */
    int32_t k_extra;    /* row width of align_ids (0 = no alignment table) */
    uint32_t flags;     /* AASD_DRAFT_* */
} aasd_draft_params;

typedef struct aasd_draft_in {
    const int32_t* hist_ids;      /* token buffers of all sequences (prompt + generated) */
    const int32_t* hist_offsets;  /* [n_seqs+1] start of each buffer; the gap is its capacity */
    const int32_t* hist_len;      /* [n_seqs] tokens currently held */
    const int32_t* prompt_len;    /* [n_seqs] how many of them are the input context */
    const int32_t* align_ids;     /* [rows x k_extra] table from aasd_align_sample, or NULL */
    const int32_t* align_n;       /* [rows] extras per table row */
    const int32_t* align_row_offsets; /* [n_seqs] table row of each sequence's first position */
    const int32_t* recent_ids;    /* [n_seqs x n] key tokens, the last recent_len[b] ... */
    const int32_t* recent_len;    /* ... of which end the current sequence (0..n) */
    /* external pool (Limitations: retrieval from a source other than the sequence itself):
       one token buffer shared by all sequences, NONE between its documents; NULL = none */
    const int32_t* pool_ids;      /* [pool_len] */
    const int32_t* pool_align_ids;/* [pool_len x k_extra] alignment table of the pool (extras of pool
                                     position q in row q - 1), or NULL */
    const int32_t* pool_align_n;  /* [pool_len] extras per row */
    int32_t pool_len;
} aasd_draft_in;

typedef struct aasd_draft_out {
    int32_t* draft_ids;    /* [n_seqs x max_cands x draft_len], NONE padded */
    uint8_t* draft_flags;  /* same shape, AASD_FLAG_* */
    int32_t* cand_len;     /* [n_seqs x max_cands] */
    int32_t* cand_pos;     /* [n_seqs x max_cands] match position of the candidate's main; a place p of
                              the external pool is reported as AASD_POOL_PLACE(p) = -2 - p */
    int32_t* n_cands;      /* [n_seqs] */
    int32_t* match_len;    /* [n_seqs] length of the matched key, 0 = no match */
} aasd_draft_out;

#define AASD_POOL_PLACE(p) (-2 - (p))

/* For every sequence: the longest k <= min(n, recent_len) such that the last k key tokens
 * occur in the history at a place that has a continuation; the places (index right after
 * the occurrence) in descending order, at most max_cands, each continued by up to
 * draft_len history tokens; then, while slots remain, alternatives in (main, depth i,
 * extra slot) order made of the main's first i tokens plus one alignment extra of position
 * p+i (extras of prompt position q are table row align_row_offsets[b] + q - 1).  All
 * outputs are required.
 * With an external pool the places of the pool compete with the history's for the longest
 * key and follow them in the list (descending within the pool); a key never matches across
 * a NONE token of the pool and a candidate ends in front of one.  Pool tokens are not input
 * context: their flag is 0 (strict verification); extras of the pool's own table are
 * alignment-sampled tokens like any other (flags 3).  The pool is scanned by every sequence's
 * CTA, so its cost grows with n_seqs x pool_len: meant for pools of up to some 10^5 tokens. */
int aasd_draft(aasd_ctx* ctx, const aasd_draft_in* in, const aasd_draft_params* params,
               const aasd_draft_out* out);

/* ---- conditional verification (Sec. 3.3, Eq. 3-6; prefix rule Sec. 2.1) ----------- */

typedef struct aasd_verify_params {
    int32_t vocab;
    int32_t dtype;
    int64_t row_stride;
    float alpha;            /* entropy factor of Eq. 5 (paper: 0.1 / 0.2) */
    float beta;             /* base threshold of Eq. 5 (paper: 0.1) */
    float inv_temperature;
    int32_t mode;           /* aasd_verify_mode */
    int32_t rows_per_cand;  /* used when cand_offsets == NULL: every candidate has this many rows */
    uint32_t step;          /* decoding step, part of the sampler's counter */
    uint64_t seed;
    int32_t top_k;          /* AASD_VERIFY_TOP_K: how many of the row's best tokens pass (>= 1) */
    uint32_t hints;         /* AASD_HINT_* */
} aasd_verify_params;

typedef struct aasd_verify_out {
    float* p_draft;       /* [n_rows] probability of the draft token (0 for NONE) */
    float* entropy;       /* [n_rows] H of Eq. 5, nats */
    float* pmax;          /* [n_rows] Delta of Eq. 6 */
    int32_t* argmax;      /* [n_rows] */
    float* threshold;     /* [n_rows] delta = min(alpha*H + beta, Delta) */
    uint8_t* accept;      /* [n_rows] accept bit of the row on its own */
    int32_t* sampled;     /* [n_rows] the row's keyed sample (STRICT_SAMPLED), else NONE */
    int32_t* accept_len;  /* [n_cands] leading accepted rows */
    int32_t* next_token;  /* [n_cands] target's own token at the first rejected row, or NONE */
    int32_t* n_greater;   /* [n_rows] AASD_VERIFY_TOP_K only: tokens ahead of the draft token in the
                             order (logit descending, id ascending); NONE for a NONE or masked
                             (-inf) draft token and on bad rows; NONE in the other modes */
} aasd_verify_out;

/* Row r holds the target distribution that judges draft_ids[r].  draft_flags may be NULL
 * (every row conditional-eligible).  A row is accepted when: CONDITIONAL mode and its flag
 * has AASD_FLAG_CONDITIONAL: p_draft >= min(alpha*H + beta, Delta), where a draft logit
 * equal to the row maximum always passes; TOP_K mode and that flag: fewer than top_k tokens
 * are ahead of it (logit descending, id ascending) and its probability is not 0; otherwise
 * draft == the target's own token (argmax, or the keyed sample in STRICT_SAMPLED).  NONE
 * never passes.  Candidates are CSR
 * row ranges (cand_offsets[n_cands+1], or regular when NULL); accept_len counts the leading
 * accepted rows and next_token is the target's own token of row accept_len if the
 * candidate has such a row.  n_rows must equal the last offset. */
int aasd_verify(aasd_ctx* ctx, const void* target_logits, const int32_t* draft_ids,
                const uint8_t* draft_flags, const int32_t* cand_offsets, int32_t n_cands,
                int64_t n_rows, const aasd_verify_params* params, void* workspace,
                size_t workspace_bytes, const aasd_verify_out* out);

/* ---- longest passing candidate (Sec. 3.3) and history update (Algorithm 1) -------- */

/* Per sequence, the candidate with the largest accept_len (ties: lowest index); emits its
 * accepted draft ids followed by its next_token when that is not NONE.  Candidates of
 * sequence b are seq_cand_offsets[b] .. seq_cand_offsets[b+1] (or cands_per_seq each when
 * the pointer is NULL); candidate c's draft ids start at cand_offsets[c] (or
 * c * rows_per_cand when NULL).  emit_ids is [n_seqs x emit_stride], NONE padded. */
int aasd_select(aasd_ctx* ctx, const int32_t* accept_len, const int32_t* next_token,
                const int32_t* draft_ids, const int32_t* cand_offsets, int32_t rows_per_cand,
                const int32_t* seq_cand_offsets, int32_t cands_per_seq, int32_t n_seqs,
                int32_t emit_stride, int32_t* best_cand, int32_t* n_emit, int32_t* emit_ids);

/* Appends the emitted tokens to each history in place (q <- q + y).  Tokens that do not
 * fit the buffer (hist_offsets[b+1] - hist_offsets[b]) are dropped and
 * AASD_STATUS_HIST_OVERFLOW is raised. */
int aasd_append(aasd_ctx* ctx, int32_t* hist_ids, const int32_t* hist_offsets,
                int32_t* hist_len, const int32_t* emit_ids, const int32_t* n_emit,
                int32_t n_seqs, int32_t emit_stride);

/* ---- one decoding step of the batched driver (Algorithm 1, loop body) ------------- */

/* aasd_step_args.flags */
#define AASD_STEP_REUSE_DRAFT 1u /* draft_out already holds this state's candidates (the caller
                                    ran aasd_draft, e.g. to feed the model): do not draft again */

#define AASD_STEP_EXTEND_TABLE 2u /* also enter the emitted tokens into the alignment table (below) */

typedef struct aasd_step_args {
    aasd_draft_in draft_in;        /* recent_ids == NULL: the key is the history's own tail */
    aasd_draft_params draft;
    aasd_draft_out draft_out;
    const void* target_logits;     /* [n_seqs*max_cands*draft_len x vocab], row = (b, c, i) */
    aasd_verify_params verify;     /* rows_per_cand is set to draft_len by the call */
    aasd_verify_out verify_out;
    int32_t* hist_ids;             /* the same buffer as draft_in.hist_ids, writable */
    int32_t* hist_len;             /* the same array as draft_in.hist_len, writable */
    int32_t* best_cand;            /* [n_seqs] */
    int32_t* n_emit;               /* [n_seqs] */
    int32_t* emit_ids;             /* [n_seqs x (draft_len+1)] */
    uint32_t flags;                /* AASD_STEP_* */
    int32_t* table_ids;            /* AASD_STEP_EXTEND_TABLE: the alignment table, writable */
    int32_t* table_n;              /*   (normally the arrays draft_in.align_ids / align_n name) */
} aasd_step_args;

/* draft -> verify -> select -> append on the context's stream (Algorithm 1, loop body), in
 * two launches: the drafting kernel, and the verification kernel, in which the warp that
 * completes a sequence's last candidate also selects and appends.  Row (b, c, i) of the
 * target logits judges token i of candidate c of sequence b, so the logits come from a
 * model run on the candidates aasd_draft emits for the same state; a caller that has just
 * made that call passes AASD_STEP_REUSE_DRAFT and the step is the second launch alone. */
int aasd_step(aasd_ctx* ctx, const aasd_step_args* args, void* workspace,
              size_t workspace_bytes);

/* Alignment sampling on generated context (AASD_STEP_EXTEND_TABLE).  The paper samples
 * extras for the input context only and names the generated context as an extension
 * (Limitations) without defining it; this is Fig. 2's rule applied to the rows the step has
 * at hand.  Row i of the winning candidate is the distribution its token i was judged
 * under, so for every emitted draft token d the extras are those of that row's
 * draft.k_extra best tokens (logit descending, ties by lower id) that rank above d - what
 * aasd_align_sample (TOPK) gives for a row whose next token is d - and the target's own
 * token that ends the emission gets none.  They go to the table row of the token's position
 * q, draft_in.align_row_offsets[b] + q - 1 (table_n, and table_ids padded with NONE), in the
 * launch that appends the token; positions beyond the history's capacity are dropped like
 * their tokens.  The table must therefore have a row for every position of every history
 * buffer (rows laid out like hist_offsets), and a caller who wants drafts to use the new
 * rows passes prompt_len = hist_len to aasd_draft.  Every verification mode (the rule does not
 * ask how a token came to be accepted), draft.k_extra 1 to AASD_MAX_EXTRA, every logits
 * layout; the workspace must have been sized by aasd_workspace_bytes. */

/* ---- draft trees (Eq. 2, Sec. 3.2) and their verification (Sec. 3.3) ---------------- */

/* Merges the candidates of every sequence (as aasd_draft writes them) into one draft tree
 * per sequence.  Tree b owns node slots [b*cap, (b+1)*cap), cap = 1 + max_cands*draft_len;
 * node 0 is the root (no token), nodes are numbered in creation order while the candidates
 * are walked in order (a parent precedes its children; children are matched by token, the
 * lowest node index first); a node reached by several candidates carries the OR of their
 * token flags.  node_parent holds indices inside the tree, NONE for the root and for unused
 * slots; node_token is NONE there too.  All outputs are required.
 * AASD_ERR_UNSUPPORTED when a tree's slots do not fit the shared memory of one CTA. */
int aasd_tree_build(aasd_ctx* ctx, const int32_t* draft_ids, const uint8_t* draft_flags,
                    const int32_t* cand_len, const int32_t* n_cands, int32_t n_seqs,
                    int32_t max_cands, int32_t draft_len, int32_t* node_token, int32_t* node_parent,
                    uint8_t* node_flags, int32_t* node_depth, int32_t* n_nodes);

typedef struct aasd_tree_out {
    float* p_token;       /* [n_rows] probability of the node's token under its parent's row (0 for roots) */
    uint8_t* accept;      /* [n_rows] the node's own accept bit (0 for roots) */
    float* entropy;       /* [n_rows] per row, as in aasd_verify_out */
    float* pmax;          /* [n_rows] */
    int32_t* argmax;      /* [n_rows] */
    float* threshold;     /* [n_rows] */
    int32_t* sampled;     /* [n_rows] the row's keyed sample (STRICT_SAMPLED), else NONE */
    int32_t* best_node;   /* [n_trees] deepest node whose whole path passes (index inside the tree;
                             the root when nothing passes; NONE for a tree without nodes) */
    int32_t* n_accept;    /* [n_trees] its depth = accepted draft tokens */
    int32_t* n_emit;      /* [n_trees] tokens in emit_ids */
    int32_t* emit_ids;    /* [n_trees x emit_stride] the tokens on the path to best_node followed by
                             the target's own token of best_node's row; NONE padded, clipped */
    int32_t* n_greater;   /* [n_rows] AASD_VERIFY_TOP_K only: tokens of the parent's row that are ahead of
                             the node's token (logit descending, id ascending); NONE for roots, NONE or
                             masked tokens, bad rows, and in the other modes */
} aasd_tree_out;

/* Verifies draft trees.  Trees are CSR ranges of nodes (tree_offsets[n_trees+1], the last
 * offset equals n_rows); row v of target_logits is the distribution that follows node v
 * given the path from the root, so the token of node v is judged with its parent's row by
 * the rules of aasd_verify (all four modes; in TOP_K mode an eligible node passes iff fewer than
 * top_k tokens of its parent's row are ahead of its token; node_flags may be NULL: every node
 * conditional-eligible).  A node passes when it and all its ancestors
 * are accepted; per tree the deepest passing node wins (ties: lowest index), which is the
 * longest candidate that passes.  Because every node has a row of its own, the token after
 * the accepted path is always available.  params->rows_per_cand is ignored.
 * A node whose parent index is not smaller than its own raises AASD_STATUS_BAD_OFFSETS and
 * never passes.  best_node, n_accept, n_emit and emit_ids are required. */
int aasd_verify_tree(aasd_ctx* ctx, const void* target_logits, const int32_t* node_token,
                     const int32_t* node_parent, const uint8_t* node_flags,
                     const int32_t* tree_offsets, int32_t n_trees, int64_t n_rows,
                     const aasd_verify_params* params, int32_t emit_stride, void* workspace,
                     size_t workspace_bytes, const aasd_tree_out* out);

/* ---- measurement aid ------------------------------------------------------------------ */

/* Reads `bytes` bytes at `buffer` (16-byte aligned, bytes a multiple of 16) once with plain
 * vector loads and folds them into *sink (4 bytes, DEVICE): no arithmetic to speak of, so the
 * time of this launch is what the device's memory system allows a read-only stream.  The
 * benchmark reports it beside the kernels' figures; it is not part of the method. */
int aasd_probe_read(aasd_ctx* ctx, const void* buffer, size_t bytes, uint32_t* sink);

/* ---- testing aid: showing that a launch whose data never arrives ends by itself -------- */

/* Every wait inside the kernels is bounded: a role that waits longer than its limit raises
 * AASD_STATUS_TIMEOUT, tells the other roles of its CTA, and all of them leave; the launch
 * then ends like any other, with invalid results for the rows concerned and a workspace that
 * has to be registered again.  This call lets a test see that happen without any fault: it
 * arms, for the NEXT launch of the streaming kernel made through this context (by
 * aasd_verify, aasd_align_sample, aasd_step or aasd_verify_tree) and for that launch only,
 *   - a wait limit of `wait_limit` polls (>= 1024) instead of the default 2^24, and
 *   - the CTA that handles work item `item` (a logits row when the call has at least twice
 *     as many rows as the device has SMs, else a piece of a row) never issuing the copy of
 *     that item's tile number `tile` (32 KB tiles, counted within the item).
 * The consumers of that CTA run out of polls, the CTA leaves, the other CTAs finish their
 * rows, and aasd_poll_status shows AASD_STATUS_TIMEOUT.  Afterwards: aasd_workspace_init on
 * the workspace, and the context works as before.  Nothing is armed when `item` lies beyond
 * the launch's items (the limit still applies).  Not for production use. */
int aasd_debug_withhold_tile(aasd_ctx* ctx, int64_t item, int32_t tile, uint32_t wait_limit);

/* ---- verification for callers that cannot allocate ------------------------------- */

#define AASD_STATIC_MAX_ROWS 8192   /* most logits rows per aasd_verify_static call */
#define AASD_STATIC_MAX_CANDS 8192  /* most candidates per aasd_verify_static call */

/* (No counterpart in the paper: this is a packaging variant of aasd_verify.)
 *
 * Some callers may not allocate device memory at the point where they verify: code that
 * runs inside a region where cudaMalloc is forbidden or would synchronise the device (an
 * inference server's steady-state loop that pre-allocated everything at start-up, a plugin
 * that only owns the buffers its host hands it, a caller holding a memory-pool lock).
 * aasd_verify needs a context (aasd_create allocates its status block) and a caller-made
 * workspace; this entry point needs neither.  Its scratch - what the workspace and the
 * context's status block would hold - lives in a fixed block of device memory that is part
 * of the library image: about 0.8 MB on every GPU that loads the library, held until the
 * process exits.  The call itself makes no cudaMalloc / cudaFree and calls nothing that
 * allocates.
 *
 * Arguments are those of aasd_verify, with the device index and the stream (a
 * cudaStream_t, NULL = legacy default stream) given directly, and results identical to
 * aasd_verify's on the same inputs.  status_bits (DEVICE pointer, may be NULL) receives the
 * AASD_STATUS_* bits this call raised, written on the stream after the kernel.
 *
 * Limits and rules:
 *  - n_rows <= AASD_STATIC_MAX_ROWS and n_cands <= AASD_STATIC_MAX_CANDS, otherwise
 *    AASD_ERR_WORKSPACE_TOO_SMALL is returned and nothing is launched.
 *  - The first call on a device looks up the block's device address (once per device, with
 *    that device made current) and so should be made before any stream capture begins.
 *  - Every call on a device shares the one block.  Each call clears the parts that must
 *    start at zero (on the stream, before its kernel), so the block's old contents never
 *    leak into a result; but two calls that can overlap on the GPU (different streams
 *    without an ordering between them) race on it and give undefined results.  Order them.
 *  - The call makes `device` the current device of the calling thread. */
int aasd_verify_static(int device, void* stream, const void* target_logits,
                       const int32_t* draft_ids, const uint8_t* draft_flags,
                       const int32_t* cand_offsets, int32_t n_cands, int64_t n_rows,
                       const aasd_verify_params* params, const aasd_verify_out* out,
                       uint32_t* status_bits);

#ifdef __cplusplus
}
#endif
#endif /* AASD_H */
