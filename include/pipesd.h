/*
 * pipesd.h -- C ABI of the cloud-side non-autoregressive verification (NAV) pass of speculative
 * decoding, implemented as hand-written CUDA kernels for sm_100a.
 *
 * The operation (paper Sec. 2.2 and Sec. 3.1 step 4): the edge sends k draft tokens; the cloud
 * validates them with ONE forward pass of the target model against the already accepted prefix,
 * accepts drafts up to the first failure, lets the target model correct that token, and -- when
 * every draft passes -- contributes one extra token (App. B).  The accepted and corrected tokens
 * become the prefix of the next round, the rejected tail is discarded (App. B).  The acceptance
 * test is the speculative-sampling rule of the works the paper builds on, which is what keeps
 * the target model's output distribution unchanged (Sec. 1): accept draft x_i while
 * u_i < min(1, p(x_i)/q(x_i)), otherwise draw from norm(max(0, p - q)).
 *
 * Conventions
 *   - Every function returns PIPESD_OK (0) or a negative pipesd_status.  Nothing throws, aborts or
 *     traps; after an error the context stays usable unless the error is PIPESD_E_CUDA.
 *   - "host" / "device" in a comment says where a pointer must live.  The library allocates no
 *     device memory: the caller provides the three device buffers sized by pipesd_query_sizes and
 *     owns them until pipesd_ctx_destroy.  The library owns small pinned host staging buffers.
 *   - All device work is enqueued on the stream given to pipesd_ctx_create (a cudaStream_t passed
 *     as void*).  A context is not thread-safe.
 *   - Model: Llama-style decoder (RMSNorm, rotary embedding with "rotate-half" pairing, grouped
 *     query attention, SwiGLU FFN, untied LM head), bf16 weights, fp32 activations, bf16 KV cache.
 *     d_model, d_ffn, vocab and the head widths must be multiples of 16; head_dim is 64 or 128.
 */
#ifndef PIPESD_H
#define PIPESD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pipesd_status {
    PIPESD_OK = 0,
    PIPESD_E_INVALID = -1,     /* null pointer, out-of-range argument, unsupported shape      */
    PIPESD_E_FULL = -2,        /* no free request slot                                        */
    PIPESD_E_OOM_PAGES = -3,   /* KV page pool exhausted; the call changed nothing            */
    PIPESD_E_STATE = -4,       /* call order violated (e.g. verify with an uncommitted tail)  */
    PIPESD_E_RANGE = -5,       /* length / count outside what the request state allows        */
    PIPESD_E_CUDA = -6,        /* a CUDA runtime call failed; see pipesd_last_error           */
    PIPESD_E_NOMEM = -7,       /* a caller-provided buffer is smaller than pipesd_query_sizes */
    PIPESD_E_TOO_LARGE = -8    /* pipesd_gemm_run_static: the problem exceeds the built-in scratch */
} pipesd_status;

#define PIPESD_MODE_STOCHASTIC 0 /* u_i < min(1, p/q), residual resample, extra token ~ p */
#define PIPESD_MODE_GREEDY 1     /* accept while draft == argmax (Sec. 2.2 prose); emit the argmax */

/* pipesd_verify flags */
#define PIPESD_Q_HOST 1u     /* item.q pointers are host memory; the library copies them on its stream.  The q arrays
                              * (like tokens, u and the results array) must then stay valid and unchanged until the
                              * next pipesd_ctx_sync returns: from pinned memory the copy is truly asynchronous */
#define PIPESD_AUTOCOMMIT 2u /* commit on the device: the kernel that takes the accept decision also writes the request's
                              * new length (base + 1 + n_accepted) and pending token to device-resident state; the host
                              * applies the same commit to its bookkeeping at the next pipesd_ctx_sync.  No
                              * pipesd_kv_rollback call follows such a verify */
#define PIPESD_CHAIN 4u      /* the cloud side of proactive transmission (App. B): this call verifies early drafts that the
                              * edge sent before it knew the outcome of the call in flight for the same requests.  They
                              * are valid iff that call accepts every draft and emits, as its extra token, this call's
                              * tokens[0]; the library plans this pass for exactly that outcome, enqueues it behind the
                              * call in flight without a host round trip, and the device decides: a pass whose condition
                              * fails returns status PIPESD_DISCARDED and commits nothing.  Implies PIPESD_AUTOCOMMIT;
                              * the call in flight must have been made with PIPESD_AUTOCOMMIT (or PIPESD_CHAIN) */

#define PIPESD_TOKEN_PENDING (-1) /* as tokens[0] of a verify item: use the pending token the library recorded for the
                                   * request (pipesd_kv_rollback's next_token, or a commit on the device) */
#define PIPESD_DISCARDED 1        /* pipesd_verify_result.status of a chained pass whose condition failed (not an error) */

typedef struct pipesd_model_cfg {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rms_eps;
    float rope_base;
    int32_t page_size;    /* tokens per KV page: a multiple of 8 (16)                          */
    int32_t n_pages;      /* pages in the pool; one page holds page_size positions of ALL layers */
    int32_t max_requests; /* request slots                                                     */
    int32_t max_draft;    /* largest k accepted by pipesd_verify (<= 31)                       */
    int32_t max_rows;     /* largest sum of (k+1) over the items of one verify call            */
    int32_t max_seq;      /* largest number of cached positions per request                    */
    int32_t device;       /* CUDA device ordinal                                               */
    int32_t reserved;     /* must be 0                                                         */
} pipesd_model_cfg;

/* Device pointers to row-major [out, in] bf16 matrices; norm gains are fp32 [d_model]. */
typedef struct pipesd_layer_weights {
    const void *wq, *wk, *wv; /* [n_q_heads*head_dim, d_model], [n_kv_heads*head_dim, d_model] x2 */
    const void *wo;           /* [d_model, n_q_heads*head_dim]                                    */
    const void *wg, *wu;      /* [d_ffn, d_model]                                                 */
    const void *wd;           /* [d_model, d_ffn]                                                 */
    const float *attn_norm, *ffn_norm;
} pipesd_layer_weights;

typedef struct pipesd_weights {
    const void *tok_emb;                /* device, bf16 [vocab, d_model]         */
    const void *lm_head;                /* device, bf16 [vocab, d_model]         */
    const float *final_norm;            /* device, fp32 [d_model]                */
    const pipesd_layer_weights *layers; /* HOST array of n_layers entries        */
} pipesd_weights;

typedef struct pipesd_sizes {
    uint64_t weights_bytes;   /* repacked weights                    */
    uint64_t kv_bytes;        /* paged bf16 KV pool                  */
    uint64_t workspace_bytes; /* activations, partial sums, metadata */
} pipesd_sizes;

/* Caller-allocated device buffers (256-byte aligned), at least as large as pipesd_query_sizes says. */
typedef struct pipesd_mem {
    void *weights; uint64_t weights_bytes;
    void *kv; uint64_t kv_bytes;
    void *workspace; uint64_t workspace_bytes;
} pipesd_mem;

/* One request of a verify call.  tokens[0] is the pending token (the previous round's correction
 * or extra token, whose KV is not cached yet), tokens[1..k] the drafts.  Row i of the forward
 * scores draft i+1; row k gives the extra-token distribution. */
typedef struct pipesd_verify_item {
    int32_t req;           /* request slot from pipesd_req_open                                  */
    int32_t k;             /* number of drafts, 1..max_draft                                     */
    int32_t mode;          /* PIPESD_MODE_*                                                      */
    int32_t reserved;
    const int32_t *tokens; /* host, k+1 ids                                                      */
    const float *q;        /* device (host with PIPESD_Q_HOST), fp32 [k, vocab] row-major draft  */
                           /* probabilities; ignored (may be null) in greedy mode                */
    const float *u;        /* host, k+1 uniforms in [0,1): u[0..k-1] acceptance tests, u[k] the  */
                           /* single final draw (correction or extra token)                      */
} pipesd_verify_item;

typedef struct pipesd_verify_result {
    int32_t n_accepted; /* 0..k                                                            */
    int32_t next_token; /* correction token if n_accepted < k, else the extra token        */
    int32_t status;     /* PIPESD_OK, PIPESD_DISCARDED, or the device-side error of the call */
    int32_t reserved;
} pipesd_verify_result;

typedef struct pipesd_ctx pipesd_ctx;

const char *pipesd_strerror(int32_t status);
/* Text of the most recent error on this context (host string owned by the context). */
const char *pipesd_last_error(const pipesd_ctx *ctx);

/* Bytes the caller must provide for a configuration.  Pure function of cfg.  (Set-up around the method: the paper's
 * cloud "only starts a server and executes NAV using the target model", Sec. 4.2, and says nothing about memory.) */
int32_t pipesd_query_sizes(const pipesd_model_cfg *cfg, pipesd_sizes *out);

/* Create a context = load the target model that performs NAV (Sec. 4.2, the target-model component of the cloud side; Sec. 5.1 for
 * the model family): validates cfg, repacks the caller's weights into mem->weights (the caller may free its own
 * weight tensors once pipesd_ctx_sync has returned), zero-initialises metadata.
 * `cuda_stream` is a cudaStream_t (null = the legacy default stream). */
int32_t pipesd_ctx_create(const pipesd_model_cfg *cfg, const pipesd_weights *w, const pipesd_mem *mem,
                          void *cuda_stream, pipesd_ctx **out);
/* Releases host state and pinned staging; the caller's device buffers are untouched. */
int32_t pipesd_ctx_destroy(pipesd_ctx *ctx);
/* Waits for the stream; delivers the results of every verify call in flight to the callers' arrays (the NAV result
 * that the cloud returns to the edge, Sec. 3.1 step 4) and applies commits made on the device to the host's
 * bookkeeping.  PIPESD_E_CUDA if a bounded device-side wait gave up since the last call: the results of the calls in
 * flight are then void (status PIPESD_E_CUDA each), nothing of them is committed, and the context stays usable. */
int32_t pipesd_ctx_sync(pipesd_ctx *ctx);

/* Request slots, one per edge device served by this cloud model (App. I: every edge is independent, one target model
 * handles the requests of all): an empty block table / return of all its pages to the pool. */
int32_t pipesd_req_open(pipesd_ctx *ctx, int32_t *req);
int32_t pipesd_req_close(pipesd_ctx *ctx, int32_t req);
/* Committed length (cached positions) of a request. */
int32_t pipesd_req_len(pipesd_ctx *ctx, int32_t req, int32_t *len);

/* Append n prompt tokens (host ids) to the request's cache -- the accepted prefix that every NAV pass runs against
 * (Sec. 2.2: the drafts are checked against the prefix accepted so far): the same layer stack as verify, run in chunks of
 * at most min(max_rows, 32) rows, no acceptance step.  If last_logits (host, vocab floats) is non-null it
 * receives the logits of the final position; the call then synchronises. */
int32_t pipesd_prefill(pipesd_ctx *ctx, int32_t req, const int32_t *tokens, int32_t n, float *last_logits);

/* The NAV pass over n_req requests in one batch (Sec. 2.2; multi-edge serving, App. I): forward of
 * each item's k+1 tokens against its cached prefix, the accept/correct rule, K/V of all k+1
 * positions written speculatively.  results (host, n_req entries) is filled when the next
 * pipesd_ctx_sync returns.  Each request must then be committed with pipesd_kv_rollback before it
 * can be verified again (PIPESD_E_STATE otherwise). */
int32_t pipesd_verify(pipesd_ctx *ctx, int32_t n_req, const pipesd_verify_item *items,
                      pipesd_verify_result *results, uint32_t flags);

/* Commit / rollback (App. B: rejected drafts are discarded, generation restarts after the last
 * accepted token): length <- base + 1 + n_accepted[i] with 0 <= n_accepted[i] <= k of the
 * request's last verify; pages wholly beyond the new length return to the pool.  No KV bytes move;
 * rows of the rejected tail are never read again.  next_token (host, n_req ids; may be null) records each
 * request's pending token -- the correction or extra token, which opens the next round's chunk (Sec. 2.2: accepted and
 * corrected tokens become the next prefix) -- so that the next verify may pass PIPESD_TOKEN_PENDING as tokens[0].
 * A request may appear once per call (PIPESD_E_INVALID otherwise; nothing is changed then).  The arguments are
 * explicit so that a harness can impose a reference decision. */
int32_t pipesd_kv_rollback(pipesd_ctx *ctx, int32_t n_req, const int32_t *reqs, const int32_t *n_accepted,
                           const int32_t *next_token);

/* ---- component entry points (used for per-kernel parity and bandwidth measurements) ---- */

/* fp32 logits [rows, vocab] of the most recent verify / prefill chunk -> host buffer. Synchronises. */
int32_t pipesd_debug_get_logits(pipesd_ctx *ctx, float *dst, int32_t rows);
/* Read / write cached K and V rows of one layer as bf16 bit patterns, host [n_pos, n_kv_heads*head_dim].
 * Writing beyond the committed length extends it (pages are allocated).  Synchronises. */
int32_t pipesd_debug_read_kv(pipesd_ctx *ctx, int32_t req, int32_t layer, int32_t pos0, int32_t n_pos,
                             uint16_t *k, uint16_t *v);
int32_t pipesd_debug_write_kv(pipesd_ctx *ctx, int32_t req, int32_t layer, int32_t pos0, int32_t n_pos,
                              const uint16_t *k, const uint16_t *v);
/* The accept/correct rule alone on caller-supplied logits (host fp32 [k+1, vocab]), q (host fp32
 * [k, vocab]), drafts (host, k ids), u (host, k+1).  Synchronises. */
int32_t pipesd_reject_from_logits(pipesd_ctx *ctx, int32_t k, int32_t mode, const float *logits,
                                  const float *q, const int32_t *drafts, const float *u,
                                  pipesd_verify_result *result);

/* Device-resident state of a request as the commit-on-device path left it: out3 (host) = {committed length, pending
 * token, 1 if the last such pass accepted every draft}.  Synchronises.  Only passes made with PIPESD_AUTOCOMMIT or
 * PIPESD_CHAIN write this state. */
int32_t pipesd_debug_req_state(pipesd_ctx *ctx, int32_t req, int32_t *out3);
/* Self-test of the error path that every bounded device-side wait of the library takes: enqueues a one-warp kernel
 * that polls a flag nothing ever sets, gives up after limit_us (1..100000) microseconds, records that in the device
 * error word and returns.  The next pipesd_ctx_sync then reports PIPESD_E_CUDA and clears the word; the context and
 * the GPU stay usable. */
int32_t pipesd_debug_wait_timeout(pipesd_ctx *ctx, int32_t limit_us);

/* Truncate a request's committed length to new_len <= its current length (pages beyond return to the
 * pool).  Lets a harness replay rounds from a recorded point; the serving path uses pipesd_kv_rollback. */
int32_t pipesd_debug_set_len(pipesd_ctx *ctx, int32_t req, int32_t new_len);

/* Launch accounting.  While enabled, every kernel launch of the context is counted and every
 * weight-streaming GEMM launch is bracketed by CUDA events on the context's stream.
 * pipesd_profile_read synchronises, reports the totals since the last read and resets them. */
typedef struct pipesd_profile_info {
    int64_t kernel_launches; /* all kernels launched by the context                         */
    int64_t gemm_launches;   /* weight-streaming GEMM launches among them                    */
    double gemm_ms;          /* summed device time of those GEMM launches (CUDA events)      */
    double gemm_bytes;       /* their algorithmic bytes: bf16 W once + fp32 x in + fp32 y out */
} pipesd_profile_info;
int32_t pipesd_profile_enable(pipesd_ctx *ctx, int32_t time_gemms);
int32_t pipesd_profile_read(pipesd_ctx *ctx, pipesd_profile_info *out);

/* Small-M weight-streaming GEMM on its own: y[M,N] = x[M,K] . W[N,K]^T with bf16 W, fp32 x and y.
 * pipesd_gemm_packed_bytes: size of the repacked copy of W (rows padded to a multiple of 128).
 * pipesd_gemm_pack: W (device, row-major bf16 [N,K]) -> packed (device).  pipesd_gemm_run: x, y device;
 * scratch device of pipesd_gemm_scratch_bytes(M,N,K) bytes (x split into bf16 hi/lo fragments; the K slices
 * are summed inside the kernel over a thread-block cluster).  N, K multiples of 16. */
uint64_t pipesd_gemm_packed_bytes(int32_t N, int32_t K);
uint64_t pipesd_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K);
int32_t pipesd_gemm_pack(const void *W, void *packed, int32_t N, int32_t K, void *cuda_stream);
int32_t pipesd_gemm_run(const void *packed, const float *x, float *y, void *scratch, int32_t M, int32_t N,
                        int32_t K, void *cuda_stream);

/* Harness switch.  Passes of more than 32 rows run their projections on the dense tensor-core kernel, smaller passes
 * on the small-M weight-streaming kernel; the two sum in different orders, so their results agree to rounding, not
 * bit for bit.  on != 0 makes every pass of the context use the dense kernel (so that a request verified alone runs the
 * projections a large batch runs; the attention's key splits still follow the pass's composition, so the two agree
 * to rounding and in their decisions, not in every bit); needs max_rows > 32 (PIPESD_E_INVALID otherwise). */
int32_t pipesd_debug_force_dense(pipesd_ctx *ctx, int32_t on);
/* CTAs of the attention kernel that the context's device keeps resident at once for a request with this many query
 * rows per KV head: out2 (host) = {with the whole third ring slot, with the cut-down one} -- the two numbers
 * pipesd_debug_attn_split takes. */
int32_t pipesd_debug_attn_slots(pipesd_ctx *ctx, int32_t rows_per_kv_head, int32_t *out2);
/* Host only, no CUDA call: how the attention kernel splits a request of `total_keys` keys (cached + this pass's
 * rows) at the given page size into CTAs that each walk tiles of 128 keys.  resident_ctas[0..1] (host) = CTAs of the
 * kernel the device keeps resident at once for the request's footprint, without and with the cut-down third slot of
 * the K/V ring; units = CTA groups that compete for the device in one layer, in groups of this request's length: KV
 * heads x row groups for a request verified alone; in a batch the batch's total of keys x groups divided by this
 * request's keys, rounded up.  out3 (host) receives {key splits, keys per split (a multiple of page_size), 1 if the
 * cut-down ring suffices}.  PIPESD_E_INVALID on bad arguments. */
int32_t pipesd_debug_attn_split(int32_t total_keys, int32_t page_size, const int32_t *resident_ctas, int32_t units,
                                int32_t *out3);

/* ---- the edge-side scheduling model (host code only; no device work) ----
 *
 * The verify pass above is what the cloud runs; what decides WHEN it runs and how the draft tokens reach it is the
 * edge's token-batch pipeline (Sec. 3.2) and its dual-threshold trigger (Sec. 3.3).  These calls make that model
 * available behind the same ABI.  Times are in any one unit (the paper uses milliseconds). */

/* T of Eq. 6 for the batching B = (b_1 = 1 < b_2 < ... < b_K <= N) of Eq. 1 (boundaries: host, K entries; b_k is the
 * index of the first draft token of batch k): with t_c = alpha + beta * n and t_ag = gamma * n for a batch of n tokens
 * (Eq. 2, 3), a batch's generation starts when the previous one's ends (Eq. 4), its transmission when both its own
 * generation and the previous transmission have ended (Eq. 5); T is the end of the last transmission.
 * PIPESD_E_INVALID if B is not such a sequence. */
int32_t pipesd_sched_round_time(int32_t N, double alpha, double beta, double gamma, const int32_t *boundaries,
                                int32_t K, double *T);
/* The batching that minimises T (Sec. 4.1, Algorithm 1; optimal by Theorem 4.1): a dynamic programme over the
 * prefixes of the N draft tokens, O(N^2).  boundaries (host, room for N entries) receives b_1..b_K, *K their number,
 * *T (nullable) the minimal time.  Among equally good batchings the one the recurrence meets first is returned. */
int32_t pipesd_sched_optimal_batching(int32_t N, double alpha, double beta, double gamma, int32_t *boundaries,
                                      int32_t *K, double *T);
/* One step of the dual-threshold trigger (Sec. 3.3) for a draft token of confidence p = P(D_n): the tentative
 * cumulative confidence is C1* = C1 * p; verification is triggered (*fire = 1) if C1* <= R1 or p <= R2.  *c1 (in/out,
 * 1 at the start) is the product over the draft tokens not yet sent to verification: it becomes 1 after a trigger
 * and C1* otherwise. */
int32_t pipesd_sched_trigger_step(double *c1, double R1, double R2, double p, int32_t *fire);

/* The same GEMM for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin or callback that is handed
 * its input and output buffers and nothing else, a real-time or latency-critical loop that must not
 * take the allocator's lock or trigger an implicit device synchronisation, a process whose memory
 * budget was fixed at start-up and has no pool to draw from.  Such callers have nowhere to get the
 * scratch that pipesd_gemm_run asks for (the activations split into bf16 fragments).  Here the scratch is a fixed array of
 * PIPESD_STATIC_SCRATCH_BYTES inside the library itself (every GPU that loads the library carries it
 * until the process ends); the call allocates and frees nothing, on the device or through any
 * library.  The caller still passes packed weights, x and y (device), exactly as for pipesd_gemm_run,
 * and gets the same result.
 *
 * Limits and rules:
 *   - If pipesd_gemm_scratch_bytes(M, N, K) is larger than PIPESD_STATIC_SCRATCH_BYTES the call returns
 *     PIPESD_E_TOO_LARGE and launches nothing.  The scratch holds 4 bytes per (token, k) with the tokens padded to
 *     whole blocks of 32 once M > 24: ceil(M/32)*32 * K * 4 bytes must fit 8 MiB, e.g. 160 rows at K=11008 (161 do
 *     not), 512 rows at K=4096.  Ask pipesd_gemm_scratch_bytes when in doubt.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and sets kernel attributes; make that first call during set-up, before any stream capture.
 *   - All calls share the one array and it keeps whatever the last call left there.  Nothing needs
 *     clearing (each call overwrites every element it later reads), but two calls whose kernels can
 *     overlap on the GPU -- different streams, no ordering between them -- race on it: keep calls on
 *     one stream or order them with events. */
#define PIPESD_STATIC_SCRATCH_BYTES (8u << 20)
int32_t pipesd_gemm_run_static(const void *packed, const float *x, float *y, int32_t M, int32_t N, int32_t K,
                               void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PIPESD_H */
