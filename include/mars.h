/*
 * mars.h -- C ABI of the B200 rollout-step library (libmars.so).
 *
 * The library computes what the paper's "Rollout module" (Section 3.3, agentic pipeline
 * parallelism; Section 2.3, segment rollouts) computes for a ragged batch of live Solver /
 * Verifier / Corrector trajectories: one forward pass of the shared policy model (a
 * Qwen3-30B-A3B-shaped mixture-of-experts decoder, Section 4.1) over the new tokens of every
 * sequence, attending over that sequence's paged key/value cache, then the sampled next token and
 * its log-probability under the behaviour policy (the denominator of the importance ratio,
 * Eq. 3).  All roles share one model and one set of sampling hyper-parameters (Section 4.1), so a
 * step has no per-role branch.
 *
 * General rules
 *   - Every byte of DEVICE memory is the caller's: weights, KV pools, workspace, metadata, inputs
 *     and outputs.  The library borrows the pointers for the lifetime of the handle that received
 *     them and owns only small host-side structures (pinned staging buffers included).
 *   - All device pointers must be 256-byte aligned unless stated otherwise.
 *   - Matrices are bf16, row-major [out_features, in_features]; norm gains are bf16 vectors.
 *   - Calls that take a stream are asynchronous on it; outputs are valid once the stream has been
 *     synchronised.  One call at a time per mars_model_t / mars_kv_t.
 *   - Errors are reported by return value only; on error nothing has been launched and the
 *     out-parameters and the cache bookkeeping are unchanged.  Token ids that are out of range on
 *     the device and bounded device-side waits that gave up are reported by mars_poll_status().
 *   - The library needs an sm_100a device; there is no CPU path.
 */
#ifndef MARS_H_
#define MARS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MARS_API __attribute__((visibility("default")))

typedef int32_t mars_status_t;
enum {
    MARS_OK = 0,
    MARS_ERR_INVALID_ARG = 1,  /* NULL / out-of-range / misaligned argument                         */
    MARS_ERR_UNSUPPORTED = 2,  /* a shape the kernels are not built for (see mars_model_load)       */
    MARS_ERR_CUDA = 3,         /* a CUDA runtime call failed (mars_last_cuda_error gives the code)   */
    MARS_ERR_KV_FULL = 4,      /* no free page / sequence already at max_pages_per_seq              */
    MARS_ERR_TIMEOUT = 5,      /* a bounded device-side wait gave up (seen by mars_poll_status)     */
    MARS_ERR_BAD_HANDLE = 6,   /* unknown sequence slot, double release, page already owned, ...    */
    MARS_ERR_BAD_TOKEN = 7,    /* a token id read on the device was outside [0, vocab)              */
    MARS_ERR_TOO_LARGE = 8     /* the request needs more than the built-in scratch array holds      */
};

/* Model shape.  max_pos bounds context_length + new tokens of any sequence. */
typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim;
    int32_t n_experts, top_k, expert_inter, vocab;
    int32_t qk_norm;   /* 1: RMS-normalise every query / key head (gain [head_dim]) before RoPE */
    int32_t max_pos;
    float rope_theta;  /* rotate-half pairing (i, i + head_dim/2), angle pos * theta^(-2i/head_dim) */
    float rms_eps;     /* inside the square root */
} mars_config_t;

/* One decoder layer; device pointers, bf16. */
typedef struct {
    const void *attn_norm;  /* [hidden]                                                    */
    const void *wqkv;       /* [(n_q + 2 n_kv) head_dim, hidden]: q rows, k rows, v rows   */
    const void *q_norm;     /* [head_dim] (ignored when qk_norm == 0)                      */
    const void *k_norm;     /* [head_dim]                                                  */
    const void *wo;         /* [hidden, n_q head_dim]                                      */
    const void *mlp_norm;   /* [hidden]                                                    */
    const void *router;     /* [n_experts, hidden]                                         */
    const void *w_gate_up;  /* [n_experts, 2 expert_inter, hidden]: gate rows, then up rows */
    const void *w_down;     /* [n_experts, hidden, expert_inter]                           */
} mars_layer_t;

typedef struct {
    const void *embed;          /* [vocab, hidden]                       */
    const void *final_norm;     /* [hidden]                              */
    const void *lm_head;        /* [vocab, hidden] (untied)              */
    const mars_layer_t *layers; /* HOST array of n_layers entries (copied by mars_model_load) */
} mars_weights_t;

/* Sampling of the next token (Section 4.1: training T 0.85 / top_p 1.0; evaluation T 0.6 /
 * top_p 0.95; top_k is always -1 in the paper and is not implemented).
 *   greedy != 0: token = argmax of the logits (lowest id on ties), log-prob at temperature 1.
 *   greedy == 0: pi = softmax(logits / temperature); nucleus = shortest prefix in (pi descending,
 *     id ascending) order with mass >= top_p; the token is drawn from pi restricted to the nucleus
 *     by inverting the cumulative distribution taken in ASCENDING TOKEN ID with one uniform per
 *     (seed, step, sequence slot) from Philox4x32-10 (key = seed, counter = (step lo, step hi,
 *     slot, 0), u = ((x0 >> 8) + 0.5) / 2^24).  The log-prob returned is log pi[token] over the
 *     full vocabulary at that temperature (the behaviour-policy probability of Eq. 3 when
 *     top_p = 1). */
typedef struct {
    float temperature, top_p;
    int32_t greedy;
    int32_t reserved;
    uint64_t seed;
    uint64_t step;
} mars_sampling_t;

/* Optional taps for tests (all device pointers, any may be NULL; NULL struct in timed runs).
 * n = number of token rows of the call (decode: n_seqs; prefill: total chunk tokens), except
 * logits, which has one row per emitted token (decode: n_seqs; prefill: requests with emit). */
typedef struct {
    float *logits;             /* [rows, vocab]                                                  */
    float *hidden;             /* [n_layers + 1, n, hidden]: residual before layer 0 / after each */
    float *router_w;           /* [n_layers, n, top_k]                                            */
    int32_t *router_idx;       /* [n_layers, n, top_k], larger probability first                  */
    const int32_t *forced_idx; /* [n_layers, n, top_k] or NULL: route to these experts instead    */
    float *nucleus_mass;       /* [rows]: probability mass of the nucleus (1 when greedy)         */
    int32_t *expert_off;       /* [n_layers, n_experts + 1]: exclusive offsets of the token permutation
                                  (expert e serves slots expert_off[e] .. expert_off[e + 1] - 1)  */
    int32_t *slot_token;       /* [n_layers, n * top_k]: token row served by every expert slot    */
} mars_debug_t;

typedef struct mars_model mars_model_t;
typedef struct mars_kv mars_kv_t;

/* Bytes of device workspace mars_model_load needs for steps of at most max_decode_seqs decode
 * sequences and max_prefill_tokens prefill tokens per call.  0 on invalid arguments. */
MARS_API size_t mars_workspace_bytes(const mars_config_t *cfg, int32_t max_decode_seqs, int32_t max_prefill_tokens);

/* Validates the shape (MARS_ERR_UNSUPPORTED unless head_dim is 64 or 128, n_q_heads / n_kv_heads
 * is an integer <= 8, hidden is a multiple of 256 in [256, 8192], expert_inter a multiple of 64 in
 * [64, 3136], top_k <= n_experts <= 1024, top_k <= 32), records the borrowed weight pointers (no copy) and carves the workspace.  The
 * workspace content is private to the library between calls. */
MARS_API mars_status_t mars_model_load(const mars_config_t *cfg, const mars_weights_t *weights, void *workspace,
                              size_t workspace_bytes, int32_t max_decode_seqs, int32_t max_prefill_tokens,
                              mars_model_t **out);
MARS_API mars_status_t mars_model_free(mars_model_t *model);

/* ---- paged KV cache -------------------------------------------------------------------------
 * Pool layout (K and V separate, bf16): [n_layers][n_pages][n_kv_heads][page_size][head_dim];
 * a page id addresses the same page in every layer.  n_pages = pool_bytes_each / bytes of one
 * layer-page / n_layers.  page_size is 16, 32, 64 or 128 tokens.  meta is device memory of
 * mars_kv_meta_bytes() bytes holding the block table [max_seqs][max_pages_per_seq] (int32). */
MARS_API size_t mars_kv_meta_bytes(int32_t max_seqs, int32_t max_pages_per_seq);
MARS_API mars_status_t mars_kv_alloc(mars_model_t *model, void *k_pool, void *v_pool, size_t pool_bytes_each,
                            int32_t page_size, int32_t max_seqs, int32_t max_pages_per_seq, void *meta,
                            size_t meta_bytes, mars_kv_t **out);
MARS_API mars_status_t mars_kv_free(mars_kv_t *kv);
MARS_API int32_t mars_kv_num_pages(const mars_kv_t *kv);
MARS_API int32_t mars_kv_free_pages(const mars_kv_t *kv);

/* Stream contract of the calls below that take no stream (reserve, adopt): the block-table entries
 * they write are on the device when the call returns (copied on a private stream of the cache and
 * waited for), so a step launched afterwards on any stream, blocking or not, sees them.  They only
 * write entries that no step in flight reads (pages appended to a slot, or an empty slot's row).
 *
 * Sequence slots 0 .. max_seqs-1.  reserve: make room for n_tokens_total tokens (allocates the
 * missing pages from the free list; MARS_ERR_KV_FULL leaves the slot unchanged).  adopt: hand the
 * slot a list of specific free pages that the caller has filled, with ctx_len tokens valid
 * (MARS_ERR_BAD_HANDLE if a page is owned already or the slot is not empty).  set_len: declare how
 * many cached tokens are valid (<= reserved capacity).  release: return the slot's pages. */
MARS_API mars_status_t mars_kv_seq_reserve(mars_kv_t *kv, int32_t seq, int32_t n_tokens_total);
MARS_API mars_status_t mars_kv_seq_adopt(mars_kv_t *kv, int32_t seq, const int32_t *pages /*host*/, int32_t n_pages,
                                int32_t ctx_len);
MARS_API mars_status_t mars_kv_seq_set_len(mars_kv_t *kv, int32_t seq, int32_t ctx_len);
MARS_API mars_status_t mars_kv_seq_release(mars_kv_t *kv, int32_t seq);
MARS_API int32_t mars_kv_seq_len(const mars_kv_t *kv, int32_t seq); /* -1 if the slot is invalid */
/* Copies the slot's page ids (host array, capacity cap) and their count. */
MARS_API mars_status_t mars_kv_block_table(const mars_kv_t *kv, int32_t seq, int32_t *pages_out, int32_t cap, int32_t *n);

/* ---- carrying a sequence across rollout segments, and forking group members --------------------
 * Rollouts are cut into fixed-length segments: a trajectory that has not finished when its segment
 * ends keeps its prefix and resumes decoding in a later segment (Section 2.3, segment rollouts).
 * A parked sequence either keeps its pages (the slot stays valid; nothing to do), or is packed into an image, released and restored later into whatever
 * pages are free then, or is dropped and its prefix fed again through mars_prefill_chunk.  All
 * three give the same next-token distribution; the first two bit for bit.
 *
 * Image layout (bf16, whole pages): [K | V][n_layers][pages of the sequence in order][n_kv_heads]
 * [page_size][head_dim]; mars_kv_seq_image_bytes(kv, n) bytes for n cached tokens (0 on a bad
 * handle).  `image` is device memory or PAGE-LOCKED host memory (the copy kernels address it
 * directly), 16-byte aligned; pageable host memory is rejected with MARS_ERR_INVALID_ARG.
 *   export: packs the slot's ceil(len / page_size) pages; asynchronous on the stream; the slot is
 *           unchanged (release it afterwards on the same stream's order to free the pages).
 *   import: the slot must be empty; reserves pages for n_tokens (MARS_ERR_KV_FULL leaves it
 *           empty), unpacks the image on the stream and sets the length to n_tokens.
 * The image must stay alive and unmodified until the stream has passed the call.
 *
 * fork: the members of a rollout group continue the same prompt (Section 3.3, grouped agentic
 * rollouts: a group of 8 outputs per selected input).  dst (empty) becomes a sequence with src's
 * cached tokens: full pages are
 * SHARED (reference-counted; a page returns to the free list when its last holder releases it), a
 * partly filled last page is copied into a fresh page on the stream, so both sequences append
 * privately.  Shared pages are never written: set_len refuses a length whose next position falls
 * into a shared page, and the step calls return MARS_ERR_BAD_HANDLE in that case.
 * mars_kv_page_refs: number of slots that list the page (0 = free, -1 = bad argument). */
MARS_API size_t mars_kv_seq_image_bytes(const mars_kv_t *kv, int32_t n_tokens);
MARS_API mars_status_t mars_kv_seq_export(mars_kv_t *kv, int32_t seq, void *image, size_t image_bytes, void *cuda_stream);
MARS_API mars_status_t mars_kv_seq_import(mars_kv_t *kv, int32_t seq, const void *image, size_t image_bytes,
                                          int32_t n_tokens, void *cuda_stream);
MARS_API mars_status_t mars_kv_seq_fork(mars_kv_t *kv, int32_t src, int32_t dst, void *cuda_stream);
MARS_API int32_t mars_kv_page_refs(const mars_kv_t *kv, int32_t page);

/* Reading a shared prefix once (on by default).  When several DECODE rows of one call list the same
 * pages from position 0 on -- the members of a rollout group after mars_kv_seq_fork (Section 3.3:
 * the outputs of a group continue one common input) -- the decode step reads the common whole pages
 * once per block of such rows instead of once per row (blocks of 16 rows on the tensor-core kernel
 * for head_dim 128 with 8 query heads per KV head, blocks of 4 rows otherwise): every K/V tile of the
 * prefix is fetched into shared memory once and scored against the queries of all rows of the block,
 * each row keeps its own online softmax, and the per-row partial results join the row's own spans in
 * the usual log-sum-exp merge.  Results equal those of the per-row reading up to fp32 summation order.
 * Prefixes shorter than 128 tokens, prompt rows, and the allocation-free entry point read per row.
 * enable == 0 switches the grouping off (every row reads its whole context), e.g. to compare. */
MARS_API mars_status_t mars_kv_share_reads(mars_kv_t *kv, int32_t enable);

/* ---- the step ---------------------------------------------------------------------------------
 * mars_decode_step: for each listed sequence slot b (context length c_b), feed in_tokens[b] at
 * position c_b, append its key/value to the cache (a new page is taken from the free list when
 * c_b is a multiple of page_size; MARS_ERR_KV_FULL is returned before anything is launched),
 * attend over positions 0..c_b, and write the sampled token and its log-prob.  c_b becomes
 * c_b + 1.  seq_ids: host, distinct.  in_tokens / out_tokens / out_logprobs: device arrays of
 * n_seqs entries; out_tokens may be passed as the next call's in_tokens.
 *
 * mars_prefill_chunk: for request r, feed chunk_lens[r] tokens (device array `tokens`, requests
 * concatenated) at positions c_r .. c_r + len - 1 with causal attention over the cache and the
 * chunk itself; c_r grows by len.  Where emit_last[r] != 0 a token is sampled from the last
 * position of the chunk; out_tokens / out_logprobs receive one entry per emitting request, in
 * request order (they may be NULL when no request emits). */
MARS_API mars_status_t mars_decode_step(mars_model_t *model, mars_kv_t *kv, void *cuda_stream, int32_t n_seqs,
                               const int32_t *seq_ids, const int32_t *in_tokens, const mars_sampling_t *sampling,
                               int32_t *out_tokens, float *out_logprobs, const mars_debug_t *debug);
MARS_API mars_status_t mars_prefill_chunk(mars_model_t *model, mars_kv_t *kv, void *cuda_stream, int32_t n_reqs,
                                 const int32_t *seq_ids, const int32_t *chunk_lens, const int32_t *tokens,
                                 const int32_t *emit_last, const mars_sampling_t *sampling, int32_t *out_tokens,
                                 float *out_logprobs, const mars_debug_t *debug);

/* mars_mixed_step: the steady state of the agentic pipeline (Section 3.3: as soon as one agent's
 * output is complete the next agent starts, so fresh Verifier / Corrector prompts arrive while
 * other trajectories are still decoding) in ONE pass per layer: n_seqs decode rows (as in
 * mars_decode_step) and n_reqs prompt chunks (as in mars_prefill_chunk) share every projection and
 * every expert contraction, so each weight is read once for both; attention runs the span kernel on
 * the decode rows and the causal kernel on the chunk rows.  Results are those of the two separate
 * calls (up to fp32 summation order).  out_tokens / out_logprobs: n_seqs entries for the decode
 * rows, then one entry per emitting request.  The slots of the two lists must be distinct.
 * Limits: n_seqs + sum(chunk_lens) <= max(max_decode_seqs, max_prefill_tokens) of mars_model_load,
 * and n_seqs + emitting requests <= max_decode_seqs. */
MARS_API mars_status_t mars_mixed_step(mars_model_t *model, mars_kv_t *kv, void *cuda_stream, int32_t n_seqs,
                                       const int32_t *seq_ids, const int32_t *in_tokens, int32_t n_reqs,
                                       const int32_t *req_ids, const int32_t *chunk_lens, const int32_t *chunk_tokens,
                                       const int32_t *emit_last, const mars_sampling_t *sampling, int32_t *out_tokens,
                                       float *out_logprobs, const mars_debug_t *debug);

/* mars_score_chunk: teacher-forced scoring of tokens that are already known -- the pass that gives
 * log pi_theta(o_t | q, o_<t) for every position of a response, i.e. the numerator of the importance
 * ratio (Eq. 3) under the current weights, or the behaviour-policy term when it is recomputed.
 * Arguments and cache effects are those of mars_prefill_chunk (the chunk tokens are appended to
 * their sequences with causal attention; several calls may score one long response chunk by
 * chunk), but nothing is sampled.  Instead, for every token row i of the call (requests
 * concatenated, as in `tokens`):
 *   out_logprobs[i] = log softmax(logits_i / temperature)[targets[i]]      when targets[i] >= 0,
 *   out_logprobs[i] = 0                                                   when targets[i] <  0
 * over the full vocabulary, where logits_i is the model output at that row's position; for a
 * response the caller passes targets[i] = the token at the next position and -1 on prompt rows and
 * on the last row.  targets, out_logprobs: device arrays of sum(chunk_lens) entries.  A target
 * >= vocab writes 0 and is reported by mars_poll_status (MARS_ERR_BAD_TOKEN).  The logits are never
 * materialised (debug->logits, if given, receives [rows, vocab] fp32; the other taps as usual).
 * MARS_ERR_UNSUPPORTED when vocab / 256 exceeds top_k * hidden / 2 (the softmax partials borrow
 * the expert-output workspace). */
MARS_API mars_status_t mars_score_chunk(mars_model_t *model, mars_kv_t *kv, void *cuda_stream, int32_t n_reqs,
                                        const int32_t *seq_ids, const int32_t *chunk_lens, const int32_t *tokens,
                                        const int32_t *targets, float temperature, float *out_logprobs,
                                        const mars_debug_t *debug);

/* Host-buffer convenience for callers that keep tokens on the host: copies in_tokens to the
 * device, runs mars_decode_step, copies the results back and synchronises the stream. */
MARS_API mars_status_t mars_decode_step_host(mars_model_t *model, mars_kv_t *kv, void *cuda_stream, int32_t n_seqs,
                                    const int32_t *seq_ids, const int32_t *in_tokens_host,
                                    const mars_sampling_t *sampling, int32_t *out_tokens_host,
                                    float *out_logprobs_host);

/* mars_decode_step_static: one decode step for callers that cannot obtain device memory of their
 * own.  (The paper has no counterpart; this entry point exists for integration reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a host
 * application that hands out the weights and the KV pools but no scratch, a real-time loop that
 * must not touch the allocator, a process whose memory pool is owned by another framework.  Such
 * callers cannot provide the workspace that mars_model_load asks for.  This call needs no handle
 * and no workspace: everything the step needs beyond its inputs and outputs (activations, split-K
 * attention partials, routing lists, logits) lives in ONE fixed array of MARS_STATIC_SCRATCH_BYTES
 * compiled into the library image.  Every GPU that loads the library carries that array until the
 * process exits.  The call itself performs no device or pinned-host allocation and frees nothing.
 *
 * Semantics are those of mars_decode_step with sequence b = block-table row b:
 *   cfg, weights      as for mars_model_load (device pointers, bf16);
 *   k_pool, v_pool    paged cache [n_layers][n_pages][n_kv_heads][page_size][head_dim], bf16;
 *   block_table       DEVICE int32 [n_seqs][max_pages_per_seq]; row b must already list the pages
 *                     that cover positions 0 .. ctx_lens[b] (nothing is taken from a free list);
 *   ctx_lens          HOST int32 [n_seqs]: tokens already cached; the new token is written at that
 *                     position and attends over 0 .. ctx_lens[b].  The caller adds 1 afterwards;
 *   in_tokens / out_tokens / out_logprobs: device arrays of n_seqs entries.
 * Limits and errors: MARS_ERR_TOO_LARGE when the step's scratch (it grows with n_seqs, vocab,
 * hidden size and cfg->max_pos) would not fit the built-in array -- nothing is launched;
 * MARS_ERR_UNSUPPORTED / MARS_ERR_INVALID_ARG as for the handle-based calls.  Token ids that are
 * out of range are read as token 0 (this call has no status word to poll).
 * First call on a device: the address of the built-in array is looked up and the kernels' launch
 * attributes are set, once per device; make that first call outside any stream capture.
 * No call may be made on a capturing stream: the step reads ctx_lens on the host and uploads its
 * work lists from host memory that is gone when the call returns, so a recorded copy would replay
 * stale data.  A stream that is capturing is refused with MARS_ERR_UNSUPPORTED before anything is
 * enqueued.
 * Sharing: all calls in the process use the same array, which keeps whatever the previous call
 * left; the call clears what must start from zero itself.  Two calls that overlap on the GPU (two
 * streams, two threads) overwrite each other's intermediates: serialise them. */
#define MARS_STATIC_SCRATCH_BYTES (4u << 20)
MARS_API mars_status_t mars_decode_step_static(const mars_config_t *cfg, const mars_weights_t *weights, void *k_pool,
                                      void *v_pool, size_t pool_bytes_each, int32_t page_size,
                                      const int32_t *block_table, int32_t max_pages_per_seq,
                                      const int32_t *ctx_lens, void *cuda_stream, int32_t n_seqs,
                                      const int32_t *in_tokens, const mars_sampling_t *sampling,
                                      int32_t *out_tokens, float *out_logprobs);

/* Precision of the dense contractions of LARGE calls (more than 256 token rows: chunked prefill, mixed
 * steps, scoring).  Activations travel as (hi, lo) bf16 pairs (~16 mantissa bits); a contraction
 * class whose bit is clear contracts the hi plane only, i.e. plain bf16 activations: half the
 * tensor-core work for ~1e-3 relative error in that contraction's output.  Decode-sized calls and the
 * lm_head always use both planes.  MARS_LO_DEFAULT is what mars_model_load sets: both planes for the QKV
 * and output projections and the router, the hi plane only for the expert contractions.  Measured on a
 * 264-token chunk through the 48-layer model against the CPU oracle (max relative L2 error of a hidden
 * state / max absolute logit error / time of an 8 x 2048-token prefill): all planes 6.4e-4 / 1.3e-3 /
 * 230 ms; QKV hi only 5.7e-3 / 8.1e-3 / 223 ms; output projection hi only 4.4e-3 / 9.0e-3 / 226 ms;
 * router hi only 1.9e-3 / 3.2e-3 / 231 ms; gate/up hi only 2.2e-3 / 3.9e-3 / 213 ms; down hi only
 * 1.8e-3 / 3.0e-3 / 221 ms; both expert contractions hi only 2.5e-3 / 3.9e-3 / 203 ms; everything hi only
 * 7.2e-3 / 1.2e-2 / 191 ms.  The default is the fastest setting that stays inside HALF of the tolerances
 * (1e-2 relative for hidden states, 2e-2 absolute for logits). */
enum {
    MARS_LO_QKV = 1, MARS_LO_OPROJ = 2, MARS_LO_ROUTER = 4, MARS_LO_GATE_UP = 8, MARS_LO_DOWN = 16,
    MARS_LO_ALL = 31,
    MARS_LO_DEFAULT = 7
};
MARS_API mars_status_t mars_set_prefill_lo_planes(mars_model_t *model, int32_t mask);

/* Synchronises the stream of the last call and reads the device status word: MARS_OK,
 * MARS_ERR_BAD_TOKEN or MARS_ERR_TIMEOUT; the word is cleared. */
MARS_API mars_status_t mars_poll_status(mars_model_t *model);

/* Self-test of the bounded device-side waits (a test hook; the paper has no counterpart).  Every
 * wait of the TMA / tensor-core kernels polls its barrier a limited number of times and, when the
 * limit is reached, sets the timeout bit of the status word, releases its tensor memory and lets the
 * kernel return.  This call launches one small block that takes exactly that path: a lane waits (at
 * most 4096 polls) for an arrival that another lane delivers when arrive != 0 and withholds when
 * arrive == 0.  With arrive == 0 the next mars_poll_status returns MARS_ERR_TIMEOUT once and the
 * handle stays fully usable; nothing hangs, traps or faults.  Asynchronous on the stream. */
MARS_API mars_status_t mars_debug_bounded_wait(mars_model_t *model, void *cuda_stream, int32_t arrive);

/* Counters of the last step call: kernels launched by it, attention work items, cached tokens read. */
typedef struct {
    int64_t kernel_launches;
    int64_t attn_items;
    int64_t kv_tokens_read; /* sum over token rows of (position + 1) */
    int64_t kv_tokens_streamed; /* cached tokens actually fetched per layer and KV head: a shared prefix
                                   counts once per block of rows, a prompt block once per block */
} mars_step_info_t;
MARS_API mars_status_t mars_last_step_info(const mars_model_t *model, mars_step_info_t *out);

/* Per-kernel-class timing for benchmarks.  While enabled, every step brackets each launch of the
 * classes below with a CUDA event pair on the step's stream (the events are host objects owned by
 * the library).  mars_profile_read synchronises the stream, adds the elapsed milliseconds and the
 * launch counts recorded since the last read into the two arrays of MARS_K_COUNT entries, and
 * recycles the events. */
enum {
    MARS_K_QKV = 0,      /* QKV projection + per-head norm + RoPE + cache append */
    MARS_K_ATTN,         /* split-K paged attention                              */
    MARS_K_ATTN_MERGE,   /* merge of the spans                                   */
    MARS_K_OPROJ,        /* output projection + residual                         */
    MARS_K_ROUTER,       /* router + permutation                                 */
    MARS_K_GATE_UP,      /* expert gate/up contraction + SwiGLU                  */
    MARS_K_DOWN,         /* expert down contraction                              */
    MARS_K_COMBINE,      /* weighted combine + residual + next norm              */
    MARS_K_LM_HEAD,      /* lm_head contraction                                  */
    MARS_K_SAMPLE,       /* log-softmax + sampling                               */
    MARS_K_OTHER,        /* step preparation, embedding                          */
    MARS_K_COUNT
};
MARS_API mars_status_t mars_profile_enable(mars_model_t *model, int32_t enable);
MARS_API mars_status_t mars_profile_read(mars_model_t *model, double *ms_per_class, int64_t *launches_per_class);

/* Device array [n_layers] (int32) inside the workspace that every step overwrites with the number
 * of distinct experts selected per layer; valid after the step's stream is synchronised. */
MARS_API const int32_t *mars_active_experts_device(const mars_model_t *model);

MARS_API int32_t mars_last_cuda_error(void);
MARS_API const char *mars_status_string(mars_status_t status);
MARS_API const char *mars_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MARS_H_ */
