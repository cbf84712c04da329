/*
 * swift.h — C boundary of the SWIFT decoding hot path on one B200 (sm_100a).
 *
 * SWIFT (arXiv 2410.06916) is self-speculative decoding with on-the-fly layer skipping: a draft
 * model made by skipping sub-layers z of the target LLM proposes tokens (Section 4.2, Eq. 4), the
 * full model verifies them in one parallel pass (Section 3.1), an acceptance rule keeps the output
 * distribution unchanged (Appendix B.2), and candidate skip sets are scored by how well they
 * re-predict the last gamma generated tokens (Section 4.1, Eq. 2-3).
 *
 * Conventions for every call
 *  - Returns a swift_status; nothing aborts, throws or traps.  swift_last_error() gives the text.
 *  - "host" / "device" on a pointer says where the memory lives.  The caller owns every buffer it
 *    passes in and keeps device buffers alive until swift_free().  The library allocates no device
 *    memory; it owns only the host-side context.
 *  - All work runs on the CUDA stream given to swift_load.  A call that returns values through host
 *    pointers synchronises that stream before returning.
 *  - On error the committed state (tokens, KV length) is unchanged.
 *  - Sub-layer masks are uint8[2*n_blocks] ordered [attn_0, mlp_0, attn_1, mlp_1, ...], 1 = skip
 *    ("L layers, including both attention and MLP layers", Section 3.1).
 *  - State machine: load -> prefill -> { draft -> verify -> accept }* ; score_skipsets and
 *    forward_rows any time after prefill when no round is open; generate = prefill + rounds.
 */
#ifndef SWIFT_H
#define SWIFT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct swift_ctx swift_ctx; /* opaque, host-side */

typedef enum {
    SWIFT_OK = 0,
    SWIFT_EINVAL = 1,       /* bad argument (null pointer, size out of range, bad token id) */
    SWIFT_ESTATE = 2,       /* call not allowed in the current state (e.g. draft before prefill) */
    SWIFT_ECAPACITY = 3,    /* rows, positions or buffer sizes beyond what was configured */
    SWIFT_ECUDA = 4,        /* a CUDA runtime call failed */
    SWIFT_ETIMEOUT = 5,     /* a bounded device-side wait ran out */
    SWIFT_EUNSUPPORTED = 6  /* shape or option this build does not handle */
} swift_status;

enum { SWIFT_F32 = 0, SWIFT_BF16 = 1 };
enum { SWIFT_GREEDY = 0, SWIFT_SAMPLING = 1 };
enum { SWIFT_MAX_ROWS = 16 }; /* rows of one forward pass: pending token + at most 15 drafts */

/* Decoder shape (LLaMA-style, the family the paper evaluates, Section 5.1). */
typedef struct {
    int32_t n_blocks, d_model, n_heads, n_kv_heads, head_dim, ffn, vocab;
    int32_t dtype;          /* SWIFT_F32 or SWIFT_BF16: storage of the weights (activations are always fp32) */
    float rope_theta, rms_eps;
    int32_t max_positions;  /* KV capacity in positions; multiple of page_size, at most 262144 */
    int32_t page_size;      /* positions per KV page; power of two, 8..128 */
    int32_t max_draft;      /* largest k any call will use; <= SWIFT_MAX_ROWS - 1 */
    int32_t kv_dtype;       /* SWIFT_F32 or SWIFT_BF16: storage of cached K,V (fp32 models: SWIFT_F32) */
} swift_model_desc;

typedef struct { void* dptr; size_t bytes; } swift_devbuf; /* caller-owned device memory, 256-byte aligned */

/* Names of the tensors swift_pack_tensor accepts.  Shapes are row-major [out_features, in_features]. */
typedef enum {
    SWIFT_T_EMBED = 0,      /* [vocab, d] */
    SWIFT_T_LM_HEAD = 1,    /* [vocab, d] */
    SWIFT_T_FINAL_NORM = 2, /* [d] fp32 gain */
    SWIFT_T_WQ = 3, SWIFT_T_WK = 4, SWIFT_T_WV = 5, /* [H*dh, d], [Hkv*dh, d], [Hkv*dh, d] */
    SWIFT_T_WO = 6,         /* [d, H*dh] */
    SWIFT_T_WGATE = 7, SWIFT_T_WUP = 8, /* [ffn, d] */
    SWIFT_T_WDOWN = 9,      /* [d, ffn] */
    SWIFT_T_ATTN_NORM = 10, SWIFT_T_MLP_NORM = 11 /* [d] fp32 gains */
} swift_tensor_kind;

/* Sizes of the three device buffers swift_load needs for this shape.  0 on an invalid desc. */
size_t swift_weights_bytes(const swift_model_desc* desc);
size_t swift_kv_bytes(const swift_model_desc* desc);
size_t swift_workspace_bytes(const swift_model_desc* desc);

/*
 * Creates a context over caller-owned device buffers.  `weights` is filled afterwards with
 * swift_pack_tensor; `kv_pool` and `workspace` need no initialisation.  `cuda_stream` is a
 * cudaStream_t (NULL = the legacy default stream).  The current CUDA device at the time of the call
 * is the device of the context.
 */
swift_status swift_load(const swift_model_desc* desc, swift_devbuf weights, swift_devbuf kv_pool,
                        swift_devbuf workspace, void* cuda_stream, swift_ctx** out);
swift_status swift_free(swift_ctx* ctx);
const char* swift_last_error(const swift_ctx* ctx); /* ctx may be NULL: last error of a failed swift_load */

/*
 * Copies one weight tensor from host memory (`src`, contiguous, the model's dtype; fp32 for gains)
 * into the library's device layout: q/k/v rows are concatenated into one fused projection, gate and
 * up rows are interleaved in groups of 16 so that one output tile holds matching gate/up pairs.
 * `block` is ignored for embed / lm_head / final_norm.  Synchronous.
 */
swift_status swift_pack_tensor(swift_ctx* ctx, swift_tensor_kind kind, int32_t block, const void* src_host,
                               size_t src_bytes);

/* Acceptance strategy for the calls that follow (Appendix B.2).  Sampling uses Philox4x32-10 keyed
 * by `seed`; temperature scales both the target's and the draft's logits.  Default: greedy. */
swift_status swift_set_sampling(swift_ctx* ctx, int32_t mode, float temperature, uint64_t seed);

/* Nucleus (top-p) filtering of the distributions sampling mode draws from and compares (the paper samples with
 * temperature 0.6 and top_p 0.95 on code generation, Appendix B.2).  Both the target's p = softmax(logits / T) and
 * the draft's q are cut to their most probable tokens whose mass first reaches top_p (every token as probable as
 * the last one included is kept) and renormalised; acceptance, the residual max(0, p - q) and the bonus draw then
 * use the cut distributions, so the output follows what plain nucleus sampling from the target would give.
 * top_p in (0, 1]; 1 (the default) = no filtering.  No effect in greedy mode.  Not allowed inside a round. */
swift_status swift_set_top_p(swift_ctx* ctx, float top_p);

/* How draft tokens are chosen in sampling mode.  0 (default): y'_j is drawn from the draft's distribution q_j and
 * accepted with probability min(1, p_j(y') / q_j(y')).  1: y'_j = argmax of the draft's logits, as Eq. 4 of Section 4.2
 * writes the drafting step; q_j is then the point mass on y'_j, so the draft is accepted with probability p_j(y') and a
 * rejected one is replaced by a draw from p_j with y'_j removed.  Both leave the output distributed as sampling from the
 * target.  No effect in greedy mode.  Not allowed inside a round. */
swift_status swift_set_greedy_draft(swift_ctx* ctx, int32_t on);

/*
 * The primitive under all three forms of the forward: M = n_rows new rows at positions
 * pos0 .. pos0+M-1 run through the sub-layers not in `skip_mask` (NULL = full model); every row
 * attends to cached positions [0, pos0) and causally to the new rows.  K,V of the new rows are
 * stored for non-skipped attention sub-layers when write_kv != 0 (positions beyond the committed
 * length stay uncommitted).  `logits_host` (may be NULL) receives n_rows*vocab fp32 values,
 * `argmax_host` (may be NULL) n_rows token ids (lowest id on ties).  pos0 <= committed length,
 * n_rows may exceed SWIFT_MAX_ROWS (processed in row chunks).  `tokens_host`: int32[n_rows].
 */
swift_status swift_forward_rows(swift_ctx* ctx, const int32_t* tokens_host, int32_t n_rows, int32_t pos0,
                                const uint8_t* skip_mask_host, int32_t write_kv, float* logits_host,
                                int32_t* argmax_host);

/* Full model over the prompt (n >= 1 tokens); caches K,V for [0, n); *first_token_host = the pending
 * token t* (argmax of the last row, or a draw from its softmax in sampling mode).  Resets the context. */
swift_status swift_prefill(swift_ctx* ctx, const int32_t* tokens_host, int32_t n, int32_t* first_token_host);

/* Replaces the pending token t* (teacher forcing: lets a caller that follows a reference sequence
 * resynchronise after a legitimate tie-break difference) and, when rounds_done >= 0, the number of
 * rounds completed so far (round r draws its random numbers at Philox counter word 0 = r, counted
 * from 1 after prefill).  Needs a prefilled context, no open round. */
swift_status swift_set_pending(swift_ctx* ctx, int32_t token, int32_t rounds_done);

/*
 * Drafting (Section 4.2, Eq. 4): up to max_k autoregressive steps of the layer-skipped model,
 * starting from the pending token at position n; token feedback and the early-stop test
 * (confidence p_j = max softmax < stop_conf; that token is kept) stay on the device.  Outputs:
 * tokens_host[max_k], conf_host[max_k] (either may be NULL), *k_host = number drafted.
 * max_k = 0 is allowed (an empty draft).  Opens a round.
 */
swift_status swift_draft(swift_ctx* ctx, const uint8_t* skip_mask_host, int32_t max_k, float stop_conf,
                         int32_t* tokens_host, float* conf_host, int32_t* k_host);

/*
 * Parallel verification (Section 3.1): the full model on rows [t*, y'_1..y'_k] at positions n..n+k,
 * writing K,V of every layer there (this fills the layers the draft skipped).  tokens_host = k draft
 * tokens, or NULL to verify what the last swift_draft produced (k is then ignored).  Outputs
 * (each may be NULL): target_argmax_host[k+1], logits_host[(k+1)*vocab].
 */
swift_status swift_verify(swift_ctx* ctx, const int32_t* tokens_host, int32_t k, int32_t* target_argmax_host,
                          float* logits_host);

/*
 * Dynamic verification (Section 4.2): with tree_rows > 0, a verification of the device's own drafts (swift_verify with
 * tokens_host == NULL, and the rounds of swift_generate) holds up to tree_rows rows instead of the drafted chain alone:
 * every draft position j is extended with the draft model's top-k predictions at that step, k = 10, 5, 3, 1 for a
 * confidence p_j in (0, 0.5], (0.5, 0.8], (0.8, 0.95], (0.95, 1].  Rows 0..k are the chain [t*, y'_1..y'_k]; the rest
 * are the alternatives, handed out from the first draft position on until the rows run out (the paper sets no limit;
 * one forward of this library holds SWIFT_MAX_ROWS rows).  An alternative of depth j sits at sequence position n + j,
 * attends to the cache, to chain rows 0..j-1 and to itself, and is stored in the cache slot of its row.  swift_accept
 * then follows, from t*, the child that equals the target's arg max, and moves an accepted alternative's K,V to the
 * slot of its depth.  Greedy decoding only (in sampling mode the setting has no effect).  tree_rows: 0 (off, the
 * default) or 2..SWIFT_MAX_ROWS.  Not allowed inside a round.
 */
swift_status swift_set_tree(swift_ctx* ctx, int32_t tree_rows);

/* Verifies a token tree the caller spells out: tokens_host[n_rows] with tokens_host[0] the pending token,
 * parent_host[n_rows] the row each row hangs off (parent_host[0] = -1, parent_host[i] < i).  Row i is stored in cache
 * slot n + i.  Outputs as swift_verify, n_rows entries.  swift_accept then walks the tree as described above. */
swift_status swift_verify_tree(swift_ctx* ctx, const int32_t* tokens_host, const int32_t* parent_host, int32_t n_rows,
                               int32_t* target_argmax_host, float* logits_host);

/* The rows of the tree the last verification held, as read back by that call (call it before swift_accept): tokens,
 * parent rows and depths, SWIFT_MAX_ROWS entries each (any may be NULL).  Returns the number of rows, 0 when the last
 * verification held a plain chain, -1 if ctx is NULL. */
int32_t swift_tree_rows(const swift_ctx* ctx, int32_t* tokens_host, int32_t* parent_host, int32_t* depth_host);

/*
 * Acceptance + KV rollback.  Greedy: a = longest prefix of drafts equal to the target's argmax,
 * next token = target argmax of row a.  Sampling: accept y'_j while u_j * q_j(y'_j) < p_j(y'_j);
 * on the first rejection the next token is drawn from max(0, p_j - q_j) renormalised, after k
 * acceptances from p_{k+1}.  Then n <- n + a + 1 and the next token becomes pending.  Closes the round.
 */
swift_status swift_accept(swift_ctx* ctx, int32_t* n_accepted_host, int32_t* next_token_host);

/*
 * Scores C candidate skip sets (Eq. 2-3): each candidate re-predicts the last gamma generated tokens
 * from their predecessors, reading the prefix K,V from the target's cache and keeping its own window
 * K,V in scratch pages.  matchness_host[C] = matches / gamma.  masks_host: uint8[C][2*n_blocks].
 * Needs gamma generated tokens (gamma <= tokens generated so far, gamma <= 128).
 */
swift_status swift_score_skipsets(swift_ctx* ctx, const uint8_t* masks_host, int32_t C, int32_t gamma,
                                  float* matchness_host);

typedef struct {
    int32_t max_new;        /* tokens to emit (exactly; there is no end-of-sequence token) */
    int32_t max_draft;      /* N_D */
    float stop_conf;        /* epsilon; 0 disables early stopping */
    int32_t vanilla;        /* 1 = plain autoregressive decoding of the full model (the baseline) */
    /* on-the-fly optimisation (Section 4.1); n_opt_rounds = 0 keeps skip_mask fixed.  An optimisation round scores the
     * set in use together with the n_candidates proposals on the last gamma generated tokens and keeps the best of them
     * (the set in use on ties, then the earliest proposal).  It ends once the kept set scores above stop_matchness,
     * after n_opt_rounds rounds, or after opt_patience rounds in a row without a replacement (0 = no such rule): the
     * stop rules of Appendix B.2. */
    int32_t gamma, n_candidates, n_opt_rounds;
    float stop_matchness;
    int32_t opt_patience;
    /* candidate_masks == NULL with n_opt_rounds > 0: the library proposes the candidates itself ("Efficient Layer Set
     * Suggestion", Section 4.1): sets of opt_skip_blocks whole blocks, uniformly random except every opt_beta-th
     * proposal (counted over the whole run), which maximises the upper confidence bound of a Gaussian-process model of
     * the scores seen so far (opt_beta 0 = random search only; the paper uses 25).  Seeded by opt_seed.  The engine and
     * what it has learnt stay with the context across calls (a stream of inputs keeps optimising one model of the
     * scores); calling with another opt_skip_blocks, opt_beta or opt_seed starts afresh. */
    int32_t opt_skip_blocks, opt_beta;
    uint64_t opt_seed;
    const uint8_t* skip_mask;       /* host, [2*n_blocks]: the (initial) draft skip set */
    const uint8_t* candidate_masks; /* host, [n_opt_rounds][n_candidates][2*n_blocks] or NULL */
} swift_gen_params;

typedef struct {
    int32_t tokens, rounds, drafted, accepted, opt_rounds, reserved;
    float best_matchness;   /* matchness of the set the last optimisation round kept (-1 if none ran) */
    float ms_prefill, ms_decode, ms_draft, ms_verify, ms_score; /* CUDA-event times on the stream */
    double bytes_draft, bytes_verify;  /* algorithmic HBM bytes of all draft / verify forwards (swift_forward_bytes, 2-byte K,V) */
    int64_t kernel_launches;           /* kernels enqueued by the whole call */
    int64_t h2d_bytes, d2h_bytes;      /* bytes the call copied host -> device and device -> host (prompt and tokens included) */
} swift_stats;

/* prefill + rounds until max_new tokens are out.  out_tokens_host[max_new]; *n_out_host = max_new.
 * `trace_host` (may be NULL) receives per round 4 int32: n_start, k, a, next_token (capacity
 * max_new rounds).  stats may be NULL. */
swift_status swift_generate(swift_ctx* ctx, const swift_gen_params* params, const int32_t* prompt_host,
                            int32_t n_prompt, int32_t* out_tokens_host, int32_t* n_out_host,
                            int32_t* trace_host, swift_stats* stats);

/*
 * The proposal engine on its own (host only, no device work): "Efficient Layer Set Suggestion" of Section 4.1.
 * swift_opt_suggest writes the next proposal as a sub-layer mask [2*n_blocks] (both sub-layers of each chosen block)
 * and, when is_bayesian_host is not NULL, whether it came from the Gaussian-process step; swift_opt_observe records
 * the matchness a mask obtained (any mask that skips whole blocks).  NULL / SWIFT_EINVAL on bad arguments.
 */
typedef struct swift_opt swift_opt;
swift_opt* swift_opt_create(int32_t n_blocks, int32_t n_skip_blocks, int32_t beta, uint64_t seed, int32_t pool);
void swift_opt_free(swift_opt* opt);
swift_status swift_opt_suggest(swift_opt* opt, uint8_t* mask_host, int32_t* is_bayesian_host);
swift_status swift_opt_observe(swift_opt* opt, const uint8_t* mask_host, float matchness);

/* Every device-side wait of this library (on a shared-memory barrier that a bulk copy or a tensor-core instruction
 * completes) is bounded: when its limit runs out the kernel records it, winds down and the next call that reads the
 * control block returns SWIFT_ETIMEOUT, with the context still usable.  This call exercises exactly that path in a
 * harmless form: one thread waits limit_us microseconds on a barrier nothing arrives on.  Returns SWIFT_ETIMEOUT
 * (that is the expected outcome); the call after it works normally. */
swift_status swift_probe_wait_limit(swift_ctx* ctx, int32_t limit_us);

/* Host-only query (no device is touched): the launch schedule of the many-row form of the tensor-core GEMM for an
 * [N][K] weight: the grid (number of persistent CTAs, at most 148) into *grid_host and the largest number of CTAs that
 * share one 128-row output tile into *max_share_host.  A chunk of many rows is bound by tensor work, so the stream-K cut
 * is chosen per shape: whole tiles per CTA where the shape has enough tiles, tiles shared between CTAs where it has few.
 * Returns SWIFT_EINVAL for null pointers or N, K < 1. */
swift_status swift_many_row_schedule(int32_t N, int32_t K, int32_t* grid_host, int32_t* max_share_host);

/* Selects the kernel behind the weight-streaming GEMMs: 1 = tensor cores (tcgen05 + TMA; default and
 * only sensible choice for bf16 models), 0 = the SIMT kernel (always used for fp32 models; for bf16 it
 * exists so that tests can check one kernel against the other).  No open round. */
swift_status swift_set_gemm_impl(swift_ctx* ctx, int32_t impl);

/* One weight-streaming GEMM of the walk on caller data: y[r][n] = sum_k x[r][k] * W[n][k] with W the
 * stored weight `which` (0 fused QKV, 1 o_proj, 2 fused gate/up in its interleaved row order, 3 down,
 * 4 output head) of `block`.  x_host: fp32 [n_rows][K], y_host: fp32 [n_rows][N].  n_rows <= 16: the kernel
 * decoding uses.  17 <= n_rows <= 512: the many-row form of the tensor-core kernel that prefill chunks and
 * side-by-side candidate scoring use, more than 128 rows as up to four row ranges ("problems") that share each weight
 * tile within one launch (bf16 models with head_dim 128 and the tensor-core kernel selected, else SWIFT_EUNSUPPORTED;
 * SWIFT_ECAPACITY if N exceeds the vocabulary size). */
swift_status swift_gemm(swift_ctx* ctx, int32_t which, int32_t block, const float* x_host, int32_t n_rows,
                        float* y_host);

/* Introspection used by tests and the benchmark. */
int32_t swift_committed_length(const swift_ctx* ctx);               /* n; -1 if ctx is NULL */
int64_t swift_launch_count(const swift_ctx* ctx);                   /* kernels enqueued since load */
/* HBM bytes one forward of n_rows rows behind n_context cached positions must move: weights of the kept sub-layers
 * and the output head, cached K,V of the kept attention sub-layers, embedding rows in, logits out.  kv_elem_bytes =
 * bytes counted per cached K or V element: 2 is what the method needs (a 16-bit cache) and what the per-round records
 * and swift_stats use; 0 counts the cache as this context stores it (4 with kv_dtype SWIFT_F32). */
double swift_forward_bytes(const swift_ctx* ctx, const uint8_t* skip_mask_host, int32_t n_rows,
                           int32_t n_context, int32_t kv_elem_bytes);
/* Per-round record of the last swift_generate on this context, for judging every forward and not only their sum
 * (the drafting stage dominates latency, paper Section 5.3; the metrics M and alpha are per round, Appendix B.3).
 * Round i (a vanilla step counts as a round with no drafts): CUDA-event time on the stream of its drafting phase
 * (all `drafted[i]` draft forwards together) and of its verification (the full-model forward plus the accept
 * step), and the algorithmic HBM bytes of those forwards.  Host arrays of `capacity` entries, any of them may be
 * NULL; returns the number of rounds recorded (which may exceed capacity; only `capacity` entries are written),
 * -1 if ctx is NULL. */
/* The skip set the last swift_generate on this context ended with: its `skip_mask` argument, or the best candidate the
 * on-the-fly optimisation kept (Section 4.1).  Feeding it to the next call as `skip_mask` is how an optimised set
 * carries over from one input to the next in a stream of inputs (the dynamic input streams of Section 5.3).
 * mask_host: [2*n_blocks] bytes, may be NULL; returns 2*n_blocks, or -1 before the first generate or if ctx is NULL. */
int32_t swift_final_skip_mask(const swift_ctx* ctx, uint8_t* mask_host);
int32_t swift_round_times(const swift_ctx* ctx, int32_t capacity, float* ms_draft_host, float* ms_verify_host,
                          double* bytes_draft_host, double* bytes_verify_host, int32_t* drafted_host);
/* The same rounds' bytes with cached K,V counted as this context stores them (swift_forward_bytes with kv_elem_bytes 0):
 * what the implementation moves, beside the algorithmic figure above.  Same conventions as swift_round_times. */
int32_t swift_round_bytes_stored(const swift_ctx* ctx, int32_t capacity, double* bytes_draft_host, double* bytes_verify_host);
/* Times `iters` back-to-back launches of one weight-streaming GEMM of the walk (which: 0 fused QKV,
 * 1 o_proj, 2 fused gate/up, 3 down, 4 output head) with n_rows rows (1..16, or 128, 256, 384 or 512: the many-row form that
 * prefill chunks and side-by-side candidate scoring use, with the plain epilogue; SWIFT_EUNSUPPORTED where the
 * model has no such form, SWIFT_ECAPACITY if the output is wider than the vocabulary), cycling over the blocks'
 * weights so that successive launches read different memory.  Outputs the average CUDA-event time per launch
 * on the stream and the weight bytes one launch streams.  Clobbers the workspace of an open round. */
swift_status swift_time_gemm(swift_ctx* ctx, int32_t which, int32_t n_rows, int32_t iters,
                             float* ms_per_launch_host, double* bytes_per_launch_host);
/* Copies K (which=0) or V (which=1) of `block` for positions [pos0, pos0+count) to host as fp32
 * [count][n_kv_heads][head_dim]. */
swift_status swift_read_kv(swift_ctx* ctx, int32_t block, int32_t which, int32_t pos0, int32_t count,
                           float* out_host);

/*
 * swift_gemm_static — the paper has no counterpart to this call; it exists for integration reasons only.
 *
 * y[r][n] = sum_k x[r][k] * w[n][k] for n_rows <= 16 rows, the same skinny weight-streaming product the
 * decoder walk is made of, for callers that are not allowed to allocate device memory: plug-ins that
 * run inside a host application which owns the allocator and hands them ready-made tensors, code that
 * runs at a point where a cudaMalloc (an implicit device synchronisation, and a lock other threads may
 * hold) is unacceptable.  The split-K partial sums and a small control block live in an array built into
 * the library image (SWIFT_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the process
 * exits), so the call allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 *  w_dev   device, row-major [N][K], SWIFT_F32 or SWIFT_BF16 (w_dtype), 16-byte aligned, K % 4 == 0
 *          (fp32) or K % 8 == 0 (bf16)
 *  x_dev   device, fp32 [n_rows][K], 16-byte aligned;   y_dev   device, fp32 [n_rows][N]
 *  All three stay the caller's.  The work is enqueued on cuda_stream (a cudaStream_t; NULL = default
 *  stream) and the call returns without synchronising.
 *
 * Limit: ceil(K / 512) * 16 * N * 4 + 1024 bytes must fit in SWIFT_STATIC_SCRATCH_BYTES, otherwise
 * SWIFT_ECAPACITY is returned and nothing is enqueued.  swift_gemm_static_error() gives the text of the
 * calling thread's last failure.
 *
 * The first call on each device looks the array's device address up (cudaGetSymbolAddress, with that
 * device current); make that first call outside any stream capture.  All calls on a device share the one
 * array and it keeps whatever the previous call left: each call re-initialises the control block and
 * overwrites every partial sum it later reads, but two calls whose kernels overlap on the GPU (different
 * streams, or concurrent host threads) race on it.  Serialise them.
 */
enum { SWIFT_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024 };
swift_status swift_gemm_static(const void* w_dev, int32_t w_dtype, int32_t N, int32_t K, const float* x_dev,
                               int32_t n_rows, float* y_dev, void* cuda_stream);
const char* swift_gemm_static_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SWIFT_H */
