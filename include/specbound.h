/*
 * specbound.h -- C ABI of the B200 (sm_100a) bounded self-speculative decode step.
 *
 * The method is SpecBound: a frozen Llama-style decoder drafts tokens from its own shallow
 * layers and verifies them with its own deep layers, producing exactly the tokens plain greedy
 * decoding would (paper: abstract; Section 3.3, last paragraph; Section 5).
 *
 * Conventions
 *   - Every function returns SB_OK (0) or a negative sb_status.  Nothing throws, aborts or traps.
 *     On error no output argument is written and the context is unchanged unless stated.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are ordinary
 *     host memory, read or written only during the call.
 *   - Device memory is BORROWED: the caller allocates and frees weights, workspace and scratch and
 *     owns the stream.  The library allocates no device memory.  sb_create pins one small host
 *     mailbox (a few KB) that sb_destroy releases.
 *   - Matrices are row-major [out_features, in_features] in the config's storage dtype, no biases,
 *     LM head untied from the embedding.  Layers are numbered 1..n_layers as in the paper.
 *   - One context = one sequence on one GPU.  A context is not thread-safe.  The stateless entry points
 *     (sb_k_*) may be called from several host threads and on several devices of one process: they
 *     serialise their host-side launch sequence internally and keep their caches per device.
 *   - Functions that return host scalars synchronise the context's stream themselves.
 *   - Device-side waits are bounded; if one expires the call returns SB_ERR_DEVICE_TIMEOUT and the
 *     CUDA context stays usable.
 */
#ifndef SPECBOUND_H
#define SPECBOUND_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sb_ctx sb_ctx;

typedef enum {
    SB_OK = 0,
    SB_ERR_ARG = -1,            /* NULL / out-of-range argument                                   */
    SB_ERR_STATE = -2,          /* call out of order (no weights, no row in flight, wrong depth)   */
    SB_ERR_CAPACITY = -3,       /* sequence, workspace or scratch too small                        */
    SB_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed                               */
    SB_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired                              */
    SB_ERR_UNSUPPORTED = -6     /* shape/dtype combination the kernels do not cover                */
} sb_status;

typedef enum { SB_F32 = 0, SB_BF16 = 1 } sb_dtype;

#define SB_MAX_W 8        /* most rows one pass may carry (w_max <= 8) */
#define SB_MAX_LAYERS 64

typedef struct {
    /* supported: n_layers <= 64, d_model <= 8192 (multiple of 8), head_dim 32 / 64 / 128, n_heads a multiple of
     * n_kv_heads with at most 4 query heads per KV head, d_ffn a multiple of 8 */
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base, rms_eps;
    int32_t dtype;   /* sb_dtype: storage of weights and of the KV cache; arithmetic is fp32 */
    int32_t max_seq; /* most positions the KV cache holds                                   */
    int32_t kv_page; /* tokens per KV page (power of two, >= 16)                            */
} sb_config;

typedef struct { /* device pointers */
    const void *attn_norm /*[d]*/, *wq /*[H*hd,d]*/, *wk /*[Hkv*hd,d]*/, *wv /*[Hkv*hd,d]*/, *wo /*[d,H*hd]*/,
        *mlp_norm /*[d]*/, *w_gate /*[F,d]*/, *w_up /*[F,d]*/, *w_down /*[d,F]*/;
} sb_layer_weights;

typedef struct {
    const void *embed /*[V,d]*/, *final_norm /*[d]*/, *lm_head /*[V,d]*/; /* device */
    const sb_layer_weights* layers;                                      /* HOST array [n_layers] */
    /* Section 3.2 trains one lightweight LM head per layer for the exit test.  Both tables are nullable HOST
     * arrays [n_layers] of DEVICE pointers, copied by sb_load_weights: exit_head[l-1] ([V,d]) replaces lm_head
     * and exit_norm[l-1] ([d]) replaces final_norm in the exit test after layer l; a NULL table or entry means
     * the shared one.  The final head of the verify pass is always lm_head / final_norm. */
    const void* const* exit_head;
    const void* const* exit_norm;
} sb_weights;

typedef struct {
    int64_t rounds, rows, accepted_drafts, emitted, probes, layer_steps, layer_row_steps;
    int64_t exit_hist[SB_MAX_LAYERS + 1]; /* [l] = rows that exited at layer l; [0] = failed by d_max */
    int64_t width_hist[SB_MAX_W + 1];     /* [w] = rounds verified with w rows                       */
    double us_prefill, us_decode;         /* host wall time around the two phases                    */
    double us_decode_dev;                 /* device time of the decode phase (CUDA events on the stream) */
    /* The next five cover the TIMED rounds only (rounds_timed of them: the first round and every fourth after it).
     * A CUDA event between two kernels keeps the later one from overlapping the earlier one's tail, so bracketing
     * every round would slow down what it measures. */
    double us_draft, us_verify;           /* device time of draft phases / of verification (alignment,
                                             unified pass, final head, acceptance)                    */
    double us_unified;                    /* device time of the unified passes alone (layers D+1..L) */
    int64_t unified_layer_steps;          /* layer passes inside us_unified                          */
    int64_t unified_kv_positions;         /* sum over those passes of the KV length they attended over */
    double us_probe_kernels;              /* device time of the exit-confidence kernels of the draft phase that were
                                             timed: one probe in 32 is bracketed by CUDA events        */
    int64_t kernel_launches;              /* kernels launched by the call                            */
    int64_t h2d_bytes, d2h_bytes;         /* bytes copied host->device / device->host by the call    */
    int64_t probes_timed;                 /* probes behind us_probe_kernels                          */
    int64_t rounds_timed;                 /* rounds behind us_draft, us_verify, us_unified           */
} sb_stats;

typedef struct { /* trace of one speculation round, filled by sb_generate when asked to */
    int32_t w, D, emitted, accepted_drafts;
    int32_t exit_layer[SB_MAX_W]; /* 0 = no exit by d_max */
    int32_t draft[SB_MAX_W];      /* -1 = none            */
    int32_t g[SB_MAX_W];          /* final greedy token of each row */
    float conf[SB_MAX_W];         /* confidence at the exit layer (or at d_max) */
} sb_round;

typedef struct {
    int32_t n;       /* positions whose KV is complete in every layer                      */
    int32_t pending; /* last committed token, not yet forwarded (-1 before prefill)         */
    int32_t rows;    /* rows in flight in the current round                                 */
    int32_t depth[SB_MAX_W];
} sb_state;

/* ---- context -------------------------------------------------------------------------------- */

/* Bytes of device workspace a context of this shape needs (KV pages + activations + scratch).
 * Returns 0 if the config is invalid. */
size_t sb_workspace_bytes(const sb_config* cfg);

/* workspace: device, >= sb_workspace_bytes(cfg), 1024-byte aligned; stays the caller's.
 * cuda_stream: a cudaStream_t (NULL = default stream) on which all work of the context runs. */
int sb_create(const sb_config* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream, sb_ctx** out);
void sb_destroy(sb_ctx* ctx);

/* Records the (device) weight pointers of a frozen base model (paper Section 4.1: the base
 * parameters are never modified) and prepares the TMA descriptors of every matrix.  The weights
 * must outlive the context.  Errors: SB_ERR_ARG (NULL / misaligned pointer: 16 bytes needed). */
int sb_load_weights(sb_ctx* ctx, const sb_weights* w);

/* Forget the sequence: n = 0, no pending token, no rows in flight.  KV pages stay allocated. */
int sb_reset(sb_ctx* ctx);
int sb_get_state(sb_ctx* ctx, sb_state* out);
/* Self-test of the bounded device-side waits: launches one small kernel that waits, for at most
 * about budget_ms (1..1000) milliseconds, on a barrier that nothing completes.  Returns
 * SB_ERR_DEVICE_TIMEOUT when the wait gave up and the kernel returned normally (the expected
 * outcome); the CUDA context stays usable, the status is cleared by the next sb_reset. */
int sb_selftest_wait_timeout(sb_ctx* ctx, int32_t budget_ms);
/* Copy the cached hidden state of in-flight row `row` (fp32 [d_model]) to host memory. */
int sb_read_hidden(sb_ctx* ctx, int32_t row, float* host_out);

/* ---- the decode step ------------------------------------------------------------------------ */

/* Prefill (Section 4.3: identical to the base model): all n_prompt tokens (host) through all
 * layers; first_token (host) receives the first generated token, which becomes `pending`. */
int sb_prefill(sb_ctx* ctx, const int32_t* prompt, int32_t n_prompt, int32_t* first_token);

/* Draft-phase primitives (Section 3.3).  push: a new row at depth 0 whose input token is `token`,
 * at position n + rows.  advance: run layers for every in-flight row whose depth is below
 * `to_layer`, lazily filling the KV of earlier rows together with the newer ones (the cache
 * manager's "Reuse"), until all rows with smaller depth reach `to_layer`. */
int sb_draft_push(sb_ctx* ctx, int32_t token);
int sb_draft_advance(sb_ctx* ctx, int32_t to_layer);

/* (a) Exit decision of Section 3.2 (Eq. 1-2) for the newest row, whose depth must equal `layer`:
 * final RMSNorm -> shared LM head -> logits / tau_l -> conf = max softmax, token = argmax,
 * exit_flag = (conf >= threshold).  One fused kernel; logits never reach HBM.  Outputs are host.
 * tau_l must be > 0 (a layer masked out of sb_generate's schedule with tau <= 0 cannot be probed:
 * SB_ERR_ARG). */
int sb_exit_confidence(sb_ctx* ctx, int32_t layer, float tau_l, float threshold, float* conf, int32_t* token,
                       int32_t* exit_flag);

/* (b) Unified parallel pass (Section 3.3; appendix "Illustration of Long Shallow Chains") over
 * the w rows in flight: alignment to the deepest row, layers D+1..L for all rows, final greedy
 * token of each row, greedy acceptance against drafts[i] (host; -1 = row i has no draft),
 * KV rollback.  out_tokens (host, [w]) receives the n_out committed tokens.  w must equal the
 * number of rows in flight. */
int sb_verify(sb_ctx* ctx, const int32_t* drafts, int32_t w, int32_t* out_tokens, int32_t* n_out);

/* Whole generation: prefill, then rounds of draft + verify until n_gen tokens are out.
 * tau (host) [d_max]: tau[l-1] = temperature T_l of layer l.  threshold: exit when conf >= it
 * (<= 0: always exit at the first probed layer; > 1: never exit).
 * Probe-layer mask: Section 3.2 tests "the first layer where p >= threshold" after every layer; on
 * this GPU a test costs a full read of the LM head (0.65 of a 7B layer's bytes), so a caller may
 * switch the test off where it rarely passes: tau[l-1] <= 0 means layer l is walked but not probed
 * (no exit can happen there; a row that reaches d_max without exiting is the difficult token as
 * usual).  The output tokens do not depend on the mask.
 * rounds (host, nullable) [max_rounds] receives the per-round trace; n_rounds (nullable) their
 * number.  stats nullable.
 * Errors: SB_ERR_ARG (d_max not in [1, n_layers-1], w_max not in [1, SB_MAX_W], NaN tau or
 * threshold, token id outside the vocabulary), SB_ERR_CAPACITY (n_prompt + n_gen + w_max > max_seq). */
int sb_generate(sb_ctx* ctx, const int32_t* prompt, int32_t n_prompt, int32_t n_gen, int32_t d_max, int32_t w_max,
                const float* tau, float threshold, int32_t* out_tokens, int32_t* n_out, sb_stats* stats,
                sb_round* rounds, int32_t max_rounds, int32_t* n_rounds);

/* Plain greedy autoregressive decoding with the same kernels (one row, all layers per token):
 * the baseline the paper's speed-ups are measured against (Section 3.4). */
int sb_generate_ar(sb_ctx* ctx, const int32_t* prompt, int32_t n_prompt, int32_t n_gen, int32_t* out_tokens,
                   int32_t* n_out, sb_stats* stats);

/* Sampling decoding (Section 4.3, "decoding strategies"; Table 2 -- the paper names temperature
 * and top-p sampling but gives no acceptance rule; this is the rule implemented).  With
 * temperature > 0, every place above that takes the full model's greedy token (sb_prefill,
 * sb_verify, sb_generate, sb_generate_ar) instead takes the inverse-CDF sample, in vocabulary
 * order, of softmax(final logits / temperature) at u = sb_sample_uniform(seed, p), p = the
 * sequence position of the token being produced (the prompt occupies 0 .. n_prompt-1): the first
 * token v whose cumulative probability reaches u.  top_p in (0, 1) restricts the distribution to
 * its nucleus first and renormalises: the tokens with logit >= z*, z* the largest logit whose
 * upper set holds at least top_p of the mass (tokens in descending probability until top_p is
 * reached; equal logits enter together); top_p = 1 keeps every token.  Drafts stay the shallow
 * layers' top-1 tokens under the annealed threshold; a draft is accepted iff it equals the
 * sampled token of its row, so sb_generate returns exactly what sb_generate_ar returns for the
 * same (temperature, top_p, seed): lossless sample by sample.  The final logits of the
 * <= SB_MAX_W rows go through a [8][vocab] fp32 buffer of the workspace and their exponentials
 * through two [8][vocab] 8-byte ones; the exit tests never write logits.  temperature 0 (the
 * default) restores greedy decoding.  Errors: SB_ERR_ARG (negative or NaN temperature, top_p
 * outside (0, 1]), SB_ERR_CAPACITY (vocab > 262144 with temperature > 0). */
int sb_set_sampling(sb_ctx* ctx, float temperature, float top_p, uint64_t seed);

/* The counter-based uniform number in (0, 1) behind sb_set_sampling: the splitmix64 output function
 * of seed + (pos + 1) * 0x9E3779B97F4A7C15, top 53 bits, centred in their cell.  Host function. */
double sb_sample_uniform(uint64_t seed, int64_t pos);

/* ---- stateless kernel entry points (micro-benchmarks, unit parity) ---------------------------- */

/* Sampling kernel alone (the rule of sb_set_sampling): token[j] (device) = inverse-CDF sample of
 * the top_p nucleus of softmax(logits[j][:] / temperature) at sb_sample_uniform(seed, pos0 + j),
 * for m <= SB_MAX_W rows of device fp32 logits [m][vocab].  scratch: device memory, 8-byte
 * aligned, at least sb_k_sample_scratch_bytes(m, vocab) bytes (the rows' exponentials, fp64 and
 * fixed point), owned by the caller.  Asynchronous on `stream` (one launch).  Errors: SB_ERR_ARG (null
 * pointer, m outside [1, SB_MAX_W], temperature <= 0, top_p outside (0, 1], scratch misaligned or
 * too small), SB_ERR_CAPACITY (vocab > 262144). */
size_t sb_k_sample_scratch_bytes(int32_t m, int32_t vocab);
int sb_k_sample(const float* logits, int32_t m, int32_t vocab, float temperature, float top_p, uint64_t seed,
                int64_t pos0, int32_t* token, void* scratch, size_t scratch_bytes, void* stream);

/* Scratch bytes the two calls below need for this shape. */
size_t sb_k_scratch_bytes(const sb_config* cfg);


/* Exit-confidence kernel on m rows of hidden states (Section 3.2, Eq. 2):
 * h device fp32 [m, d]; final_norm / lm_head device in cfg->dtype; tau_l > 0.
 * conf device fp32 [m], token device int32 [m]; logits_dbg nullable device fp32 [m, vocab]
 * (debug dump only).  scratch: device, >= sb_k_scratch_bytes, 1024-byte aligned. */
int sb_k_exit_confidence(const sb_config* cfg, const void* h, int32_t m, const void* final_norm, const void* lm_head,
                         float tau_l, float* conf, int32_t* token, float* logits_dbg, void* scratch,
                         size_t scratch_bytes, void* cuda_stream);

/* The same exit-confidence computation for callers that cannot allocate device memory (the paper has
 * no counterpart; this is a convenience of the library).  Some users of this kernel run where
 * cudaMalloc is off limits -- inside a serving loop whose memory was handed out once at start-up,
 * under a framework that owns the caching allocator and forbids foreign allocations, or in a
 * latency-critical path where an allocation's implicit synchronisation is unacceptable -- and they
 * have no spare buffer to lend as scratch.  This variant takes none: its scratch is a fixed 1 MiB
 * array in device memory that every GPU holding the library keeps from load to exit.
 *   - Inputs and outputs are still the caller's: h device fp32 [m, d], final_norm / lm_head device
 *     in cfg->dtype, conf device fp32 [m], token device int32 [m]; work runs on cuda_stream.
 *   - Limit: the rows, their normalised copy and the per-CTA partial results must fit the array,
 *     which holds for d_model <= 8192; a larger model is refused with SB_ERR_CAPACITY.  Other
 *     errors as sb_k_exit_confidence (SB_ERR_ARG for bad pointers, m outside 1..8, tau_l <= 0).
 *   - The call allocates nothing on the device: no cudaMalloc / cudaFree, no allocating library
 *     routine.  The first call on each device looks up the array's device address (a short
 *     host-side query); make that first call before any stream capture starts.
 *   - All calls on one device share the array and it keeps the previous call's contents; the call
 *     itself resets the words that must start at zero.  Two calls whose GPU work overlaps (different
 *     streams, or different host threads) race on it: serialise them. */
int sb_k_exit_confidence_static(const sb_config* cfg, const void* h, int32_t m, const void* final_norm,
                                const void* lm_head, float tau_l, float* conf, int32_t* token, void* cuda_stream);

/* One decoder layer for m rows at positions first_pos .. first_pos+m-1 (the verify pass of one
 * layer, Section 3.3): h device fp32 [m, d] in/out.  k_cache / v_cache: device, cfg->dtype,
 * [n_pages, kv_page, n_kv_heads*head_dim]; page_table device int32 [ceil(max_seq / kv_page)]
 * maps logical page -> physical page.  Appends K,V of the m rows, attends causally over
 * positions 0 .. own position. */
int sb_k_layer(const sb_config* cfg, const sb_layer_weights* lw, void* h, int32_t m, void* k_cache, void* v_cache,
               const int32_t* page_table, int32_t first_pos, void* scratch, size_t scratch_bytes, void* cuda_stream);

/* The same for n_layers consecutive layers in one launch sequence (the steady state of the verify
 * pass, Section 3.3: the weights of the layers D+1..L streamed back to back): layer i uses lw[i],
 * k_caches[i], v_caches[i] (HOST arrays [n_layers]; the caches are device memory laid out as for
 * sb_k_layer and share page_table).  rope_table: nullable device table of the rotation angles made
 * by sb_k_rope_table for this config (without it every launch computes its angles).  One status
 * clear at the start, then every kernel overlaps its predecessor's tail as inside sb_generate. */
size_t sb_k_rope_table_bytes(const sb_config* cfg);
int sb_k_rope_table(const sb_config* cfg, void* table, size_t table_bytes, void* cuda_stream);
int sb_k_layer_chain(const sb_config* cfg, const sb_layer_weights* lw, int32_t n_layers, void* h, int32_t m,
                     void* const* k_caches, void* const* v_caches, const int32_t* page_table, int32_t first_pos,
                     const void* rope_table, void* scratch, size_t scratch_bytes, void* cuda_stream);

/* ---- helpers ---------------------------------------------------------------------------------- */

/* Eq. 1: out[l-1] = 1 + alpha (1 - l/L) for l = 1..L (host). */
int sb_tau_schedule(float alpha, int32_t L, float* out);
/* Eq. 5: analytic speed-up for acceptance rate a, draft width w, depth bound d_max. */
double sb_model_speedup(int32_t L, double a, int32_t w, int32_t d_max);

/* Options.
 *   SB_OPT_GEMM      0 = CUDA-core streaming kernels, 1 = TMA + tcgen05 kernels (bf16 only).
 *   SB_OPT_TRACE     (default option only) 1 = sb_k_layer times each of its launches with CUDA events
 *                    and prints them to stderr; a profiling aid, off by default.
 *   SB_OPT_TC_TUNING (default option only) stages * 16 + CTAs per SM of the tcgen05 kernels.
 *   SB_OPT_PDL       (default option only) 1 (default) = launch kernels with programmatic dependent
 *                    launch so that a kernel's prologue and weight prefetch overlap its predecessor.
 *   SB_OPT_L2_PREFETCH (default option only) n > 0: while the output projection waits for the attention
 *                    kernels (HBM idle), it prefetches every n-th k block of the layer's gate/up weights
 *                    into L2; 0 = off.  Default 4.  Needs bit 0 of SB_OPT_FUSE.
 *   SB_OPT_SPLIT_PENALTY (default option only) what the work decomposition charges per additional k split,
 *                    in per mille of the streaming time (more splits balance the CTAs better but cost
 *                    partial-sum traffic and consumer loads).
 *   SB_OPT_FUSE      (default option only) bit mask, default 3.
 *                    1: the tcgen05 gate/up GEMM pairs gate and up rows in one tile and its epilogue writes
 *                       SwiGLU as the down projection's operand (otherwise SwiGLU is a kernel of its own).
 *                       The fused GEMM is never split along k, so its sums may round differently from the
 *                       separate kernels' (fp32 rounding level).
 *                    2: RoPE, KV-cache append and attention run inside the attention kernel: up to 8 chunks of 128
 *                       positions in one launch whose chunk CTAs form a
 *                       thread-block cluster and merge the chunks; longer contexts in two (chunk kernel, chunk merge).
 *                       Off: three launches (RoPE/append, chunk kernel, chunk merge).  Bit-identical either way.
 *                    Each setting by itself is deterministic and row-invariant.
 *   SB_OPT_QKV_AHEAD (default option only) 1 (default) = while sb_generate waits for an exit decision it already
 *                    issues the RMSNorm and QKV GEMM of the layer step that follows if the row does not exit
 *                    (they write scratch only; on an exit they are discarded).  Results do not depend on it.
 *   SB_OPT_WIDE_PREFILL (default option only) 1 (default) = sb_prefill of a bf16 model on the tcgen05 path (with the
 *                    SwiGLU epilogue on) sends up to 128 prompt rows per pass through the weight-streaming GEMMs (the
 *                    weights are read once per 128 rows), with a tiled causal attention kernel on the tensor cores, and
 *                    the fewer than 16 rows left over through 8-row passes; 2 = the same passes with the decode attention
 *                    kernels (a block of 8 rows at a time); 3 = as 1, but every work item of a wide GEMM on one CTA instead of
 *                    a pair of CTAs sharing one activation tile; 0 = 8-row passes only.  All are deterministic; they may differ
 *                    in summation order, i.e. in the last bits of the K/V cache and of the first token's logits. */
enum { SB_OPT_GEMM = 1, SB_OPT_TRACE = 2, SB_OPT_TC_TUNING = 3, SB_OPT_PDL = 4, SB_OPT_L2_PREFETCH = 5,
       SB_OPT_SPLIT_PENALTY = 6, SB_OPT_FUSE = 7, SB_OPT_QKV_AHEAD = 8, SB_OPT_WIDE_PREFILL = 9 };
int sb_set_option(sb_ctx* ctx, int32_t key, int32_t value);

/* Process-wide default for contexts and stateless calls created afterwards. */
int sb_set_default_option(int32_t key, int32_t value);

/* The work decomposition the weight-streaming GEMMs of a layer pass use (Section 3.3: the skinny-M GEMMs of the draft
 * steps and of the unified pass; Section 4.3: prefill).  Host arithmetic only: no device is touched, nothing is launched;
 * meant for tests and for sizing studies.
 *   mode 0: the 8-row kernel on `units` CTAs; 1: its gate/up form (n_rows[0] = FFN width, n_mats = 1);
 *   mode 2: the 128-row kernel on `units` clusters of two CTAs; 3: its gate/up form.
 *   n_rows[n_mats] (1..3 matrices that share k and the activation operand, HOST array), k = inner dimension.
 * Out (HOST): rows_per_cta = weight rows a CTA stages per work item (gate/up: FFN columns per item), k_splits, n_items =
 * slabs x splits.  Returns SB_ERR_ARG for null pointers, mode outside 0..3, n_mats outside 1..3 or non-positive sizes. */
int sb_plan_gemm(int32_t mode, const int32_t* n_rows, int32_t n_mats, int32_t k, int32_t units, int32_t* rows_per_cta,
                 int32_t* k_splits, int32_t* n_items);

const char* sb_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SPECBOUND_H */
