/*
 * libasd -- adaptive self-speculative decoding (arXiv 2410.01028) on one NVIDIA B200 (sm_100a).
 *
 * The library runs single-sequence, memory-bound decoding of a Llama-style dense decoder M in which
 *   - every attention and MLP sublayer of a full-model pass also yields the cosine similarity between the
 *     hidden state entering and leaving it (Section 3.1; the summand of C_l in Section 3.2), computed in the
 *     epilogue of the residual add;
 *   - the Adaptive Draft Model Generator (Algorithm 1; rules 1 and 2 of Section 3.2) turns the similarities
 *     averaged over the prompt into a per-context skip mask that defines the draft model D, a sub-network of M;
 *   - k drafted tokens are verified by one (k+1)-row pass of M, the matching prefix is accepted and the first
 *     rejected token is replaced by M's (Section 1), so the output equals greedy autoregressive decoding.
 *
 * Conventions
 *   - C ABI. Every call returns an int: ASD_OK (0) or a negative asd_status. No call throws or aborts;
 *     asd_last_error() returns a description of the last failure of that context (static storage duration
 *     per context; valid until the next failing call).
 *   - Pointers are HOST pointers unless the parameter is documented as DEVICE. Host arrays are borrowed for
 *     the duration of the call only. Calls are synchronous with respect to their host outputs.
 *   - The context owns no device memory: all of it is carved out of one caller-provided DEVICE workspace of
 *     asd_workspace_bytes() bytes (256-byte aligned), which must outlive the context. Work is enqueued on
 *     the caller-provided CUDA stream (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - One context holds one sequence (batch size 1, as in Section 3.2). Contexts are not thread safe.
 *   - Layers are numbered l = 1..L in the paper; arrays indexed by layer use index l-1.
 *   - Matrices are bf16, row-major [out, in] (y = W x); accumulation is fp32; the residual stream is fp32.
 */
#ifndef ASD_H_
#define ASD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ASD_OK = 0,
    ASD_ERR_ARG = -1,            /* null pointer, out-of-range value, unsupported shape */
    ASD_ERR_STATE = -2,          /* call not valid in the current state (no weights, nothing prefetched, ...) */
    ASD_ERR_NOMEM = -3,          /* workspace too small or misaligned */
    ASD_ERR_OVERFLOW = -4,       /* the call would write past max_seq positions */
    ASD_ERR_CUDA = -5,           /* a CUDA runtime call failed; see asd_last_error() */
    ASD_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired */
    ASD_ERR_IO = -7              /* weight file missing, short or malformed */
} asd_status;

/* Shape of the decoder. Requirements: n_heads * head_dim == d_model; n_heads % n_kv_heads == 0;
 * head_dim in {16, 32, 64, 128, 256}; d_model % 8 == 0; d_ffn % 8 == 0; 0 <= max_draft <= 8. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t max_seq;   /* capacity of the KV cache in positions */
    int32_t max_draft; /* largest draft length k accepted by asd_verify / asd_generate */
    float rms_eps;     /* epsilon under the root of RMSNorm */
    float rope_theta;  /* base of the rotary embedding */
} asd_config;

/* bf16 weights on the HOST, as raw 16-bit patterns, row-major [out, in], stacked over layers. */
typedef struct {
    const uint16_t* embed;      /* [vocab, d_model]                 */
    const uint16_t* lm_head;    /* [vocab, d_model] (untied)        */
    const uint16_t* final_norm; /* [d_model]                        */
    const uint16_t* attn_norm;  /* [L, d_model]                     */
    const uint16_t* wq;         /* [L, d_model, d_model]            */
    const uint16_t* wk;         /* [L, n_kv_heads*head_dim, d_model]*/
    const uint16_t* wv;         /* [L, n_kv_heads*head_dim, d_model]*/
    const uint16_t* wo;         /* [L, d_model, d_model]            */
    const uint16_t* mlp_norm;   /* [L, d_model]                     */
    const uint16_t* wg;         /* [L, d_ffn, d_model]  gate        */
    const uint16_t* wu;         /* [L, d_ffn, d_model]  up          */
    const uint16_t* wd;         /* [L, d_model, d_ffn]  down        */
} asd_host_weights;

/* Hyper-parameters of Algorithm 1. flags select the rule subsets of Table 5. */
#define ASD_USE_CS 1u    /* cosine-similarity thresholding: remove attention layer l if C_l >= alpha */
#define ASD_USE_RULE1 2u /* remove every m-th attention and MLP layer */
#define ASD_USE_RULE2 4u /* never remove the last n layers */
#define ASD_ADMG_ALL 7u
/* Two extensions that the paper does not have, both off unless their flag is set:
 *   ASD_USE_CS_MLP  Table 1 measures the MLP similarities but Algorithm 1 never looks at them. With this flag an MLP
 *                   layer l <= L - n is also removed when its own C_l reaches alpha_mlp (remove_ATTN is unchanged).
 *   ASD_RUNNING_C   Section 3.2 computes C_l over the prompt only. With this flag every row that a full-model pass
 *                   commits after the prompt (decode steps, the accepted rows of a verify pass) joins the mean, and
 *                   asd_generate runs Algorithm 1 again on the refreshed C_l every `refresh` rounds (0 = never). */
#define ASD_USE_CS_MLP 8u
#define ASD_RUNNING_C 16u
typedef struct {
    float alpha;
    int32_t m, n;
    uint32_t flags;
    float alpha_mlp; /* threshold of ASD_USE_CS_MLP; ignored without that flag */
    int32_t refresh; /* rounds between mask updates under ASD_RUNNING_C; ignored without that flag */
} asd_admg_params;

#define ASD_MODE_AR 0               /* plain greedy decoding with M */
#define ASD_MODE_SPEC 1             /* self-speculative; mask from Algorithm 1 on the prompt's similarities */
#define ASD_MODE_SPEC_MANUAL_MASK 2 /* self-speculative with the mask installed by asd_set_skip_mask */
typedef struct {
    int32_t mode, draft_len, max_new;
    int32_t eos_id; /* -1 = none */
    asd_admg_params admg;
    /* Draft exiting (Section 4 takes the mechanism from Draft & Verify without restating it; this is its fixed-threshold
     * form): a round stops drafting after the first draft token whose confidence in the draft model D, measured as
     * the gap between D's largest and second-largest logit, is below this value; that token is still verified.
     * 0 = off (every round drafts draft_len tokens). Costs one host read-back per draft step. */
    float draft_exit_margin;
    /* Sampling (Section 1; the T > 0 columns of Tables 3 and 4): 0 = greedy decoding as described above. Above 0 every
     * token is drawn from softmax(logits / temperature) and the verification accepts drafts so that the output keeps
     * the full model's distribution; see asd_set_sampling for the rule and the random numbers. */
    float temperature;
    uint64_t seed;
} asd_gen_params;

/* Counters and device times (CUDA events) accumulated since the last asd_reset / asd_generate start.
 * bytes_* are the algorithmic bytes of the passes: weights actually streamed plus K/V read. */
typedef struct {
    int64_t full_passes, draft_passes, verify_passes, rounds, drafted, accepted, prefill_rows;
    double ms_prefill, ms_full, ms_draft, ms_verify, ms_total;
    double bytes_full, bytes_draft, bytes_verify;
    int64_t kernel_launches;
} asd_stats;

typedef struct asd_ctx asd_ctx;

/* Size of the device workspace a context of this shape needs (weights + KV cache + scratch); 0 on a bad config.
 * Where the tensor-core prompt path is available (head_dim 64 or 128) every sublayer matrix is kept twice, once in the
 * packed order the decode passes stream and once row-major for the prompt GEMMs: about twice the bf16 weights, e.g.
 * ~27 GB for the 7B shape and ~52 GB for the 13B shape before the KV cache, whatever asd_set_prefill_mode selects
 * later. The packed copy is cut into one slab per SM of the device that is current when the weights are loaded, so
 * a workspace image is not portable between devices with different SM counts. */
size_t asd_workspace_bytes(const asd_config* cfg);

/* Create a context inside dev_workspace (DEVICE, 256-byte aligned, >= asd_workspace_bytes(cfg)).
 * The workspace's KV region is zeroed. cuda_stream is a cudaStream_t. Errors: ARG, NOMEM, CUDA. */
int asd_create(const asd_config* cfg, void* dev_workspace, size_t bytes, void* cuda_stream, asd_ctx** out);
int asd_destroy(asd_ctx* ctx);
const char* asd_last_error(asd_ctx* ctx);

/* Copy the weights into the workspace, repacked into the order in which the pass kernel streams them. Blocking. */
int asd_load_weights_host(asd_ctx* ctx, const asd_host_weights* w);
/* Same tensors from a flat little-endian file: the twelve arrays of asd_host_weights in declaration order,
 * without header or padding. Errors: IO when the file is missing or short. */
int asd_load_weights_file(asd_ctx* ctx, const char* path);

/* New context: nothing cached, similarity sums cleared, empty skip mask, statistics cleared. */
int asd_reset(asd_ctx* ctx);

/* Section 3.2, first step of inference: pass n prompt tokens through M, fill the KV cache, add each row's
 * per-sublayer cosine to the running sums behind C_l, return M's first token. May be called again to append
 * more prompt. Errors: ARG (n <= 0, token out of range), OVERFLOW, STATE (no weights). */
int asd_prefill(asd_ctx* ctx, const int32_t* tokens, int32_t n, int32_t* first_token);
/* As asd_prefill with the tokens in DEVICE memory (inputs already resident). */
int asd_prefill_device(asd_ctx* ctx, const int32_t* dev_tokens, int32_t n, int32_t* first_token);

/* C_l of Section 3.2 for the attention sublayers (c_attn[L]) and, as in Table 1, the MLP sublayers
 * (c_mlp[L]); n_rows = number of prompt rows averaged. Any output may be NULL. STATE if no row yet. */
int asd_get_similarity(asd_ctx* ctx, float* c_attn, float* c_mlp, int32_t* n_rows);

/* Algorithm 1 on the current C: computes remove_ATTN / remove_MLP, installs them as the draft model's skip
 * mask and optionally returns them (uint8[L], 1 = removed). Resets the draft cursor. */
int asd_admg_update(asd_ctx* ctx, const asd_admg_params* p, uint8_t* skip_attn, uint8_t* skip_mlp);
/* Turns the running similarities (ASD_RUNNING_C, see asd_admg_params) on or off for the single-step calls:
 * while on, asd_decode_step adds its row and asd_verify its a+1 committed rows to the sums behind C_l.
 * asd_generate sets it from its parameters' flags. asd_reset leaves it as it is. */
int asd_set_running_similarity(asd_ctx* ctx, int32_t on);
/* Install a mask by hand (uint8[L] each, non-zero = skip). Resets the draft cursor. */
int asd_set_skip_mask(asd_ctx* ctx, const uint8_t* skip_attn, const uint8_t* skip_mlp);

/* One autoregressive step of M: consumes token_in at the next position, commits it, returns the argmax. */
int asd_decode_step(asd_ctx* ctx, int32_t token_in, int32_t* token_out);
/* One step of the draft model D at the draft cursor: sublayers in the mask are the identity, stream no
 * weights and touch no K/V. Commits nothing; advances the draft cursor. */
int asd_draft_step(asd_ctx* ctx, int32_t token_in, int32_t* token_out);
/* Section 1: M processes tokens[0..k] = [t_last, d_1..d_k] at the next k+1 positions in one pass, rewriting
 * K/V there in every layer. d_{j+1} is accepted while it equals M's argmax g_j; out_tokens receives the
 * accepted drafts followed by g_a (a+1 tokens, a = *n_accepted); a+1 positions are committed and the draft
 * cursor returns to the committed length. 0 <= k <= max_draft. */
int asd_verify(asd_ctx* ctx, const int32_t* tokens, int32_t k, int32_t* n_accepted, int32_t* out_tokens);

/* Decoding with sampling instead of the argmax (Section 1 on verification "when sampling is used", which points to
 * the rule of speculative sampling; the paper runs T = 0.2 and T = 0.6 in Tables 3 and 4). temperature = 0 restores
 * greedy decoding. With temperature > 0:
 *   - asd_prefill's first token and asd_decode_step's token are drawn from p = softmax(logits / temperature);
 *   - asd_draft_step draws its token from the draft model's distribution q and keeps q on the device;
 *   - asd_verify takes the tokens drawn by this round's draft steps (anything else: ASD_ERR_STATE) and accepts draft x
 *     at a position when its uniform number r satisfies r < min(1, p(x)/q(x)); the first rejected draft is replaced
 *     by a draw from max(0, p - q) normalised, and a round in which all drafts are accepted ends with one more draw
 *     from p. Every emitted token is then distributed as if M had drawn it.
 * Random numbers: the counter-based generator Philox4x32-10 with key = seed and counter = (position of the token being
 * chosen, kind of draw: 0 draft, 1 acceptance test, 2 full model's draw, 0, 0); its first output word x gives the
 * uniform number (x + 1/2) / 2^32. Probabilities and all comparisons are evaluated in double precision on the device.
 * asd_generate takes both values from its parameter block instead. Errors: ARG (negative or NaN temperature). */
int asd_set_sampling(asd_ctx* ctx, float temperature, uint64_t seed);

/* The whole method: reset, prefill, t_1, (Algorithm 1), then rounds of draft_len draft steps and one verify
 * until max_new tokens (out[0] = t_1) or eos. out has room for max_new tokens. stats may be NULL. */
int asd_generate(asd_ctx* ctx, const int32_t* prompt, int32_t n_prompt, const asd_gen_params* p, int32_t* out,
                 int32_t* n_out, asd_stats* stats);
/* As asd_generate with the prompt and the output array in DEVICE memory; n_out stays a host pointer. */
int asd_generate_device(asd_ctx* ctx, const int32_t* dev_prompt, int32_t n_prompt, const asd_gen_params* p,
                        int32_t* dev_out, int32_t* n_out, asd_stats* stats);

/* How asd_prefill (and the prefill inside asd_generate) processes the prompt, the first step of inference in
 * Section 3.2. Either way it fills the KV cache, adds every prompt row's per-sublayer cosine similarity to the
 * sums behind C_l and returns t_1.
 *   ASD_PREFILL_ROWS  passes of up to 16 rows through the decode kernel: row r of the prompt is bit-identical to
 *                     a one-row pass at the same position.
 *   ASD_PREFILL_GEMM  all rows as dense bf16 products on the tensor cores (fp32 accumulation, the same rounding
 *                     points; the accumulation order differs, so results agree with ASD_PREFILL_ROWS to
 *                     rounding, not bit for bit), then the LM head alone on the last row's hidden state.
 *                     Needs head_dim 64 or 128, else ASD_ERR_ARG.
 *   ASD_PREFILL_AUTO  (default) ASD_PREFILL_GEMM for prompts of more than 32 tokens where the shape allows it,
 *                     otherwise ASD_PREFILL_ROWS.
 * After a prompt that took the dense path, asd_get_last_cosines / asd_get_last_logits describe the last prompt
 * token (one row). */
#define ASD_PREFILL_AUTO 0
#define ASD_PREFILL_ROWS 1
#define ASD_PREFILL_GEMM 2
int asd_set_prefill_mode(asd_ctx* ctx, int32_t mode);

/* Per-row results of the last pass of M rows: cosines [L][M] (NaN where the sublayer was skipped),
 * argmax [M]. *M receives the row count. Any output may be NULL. */
int asd_get_last_cosines(asd_ctx* ctx, int32_t* M, float* cos_attn, float* cos_mlp);
/* Top-2 logit gap (largest minus second-largest logit; 0 when two tokens tie) of every row of the last pass that
 * ran the LM head, margins[M]. margins may be NULL to query M. Errors: STATE if no such pass has run. */
int asd_get_last_margins(asd_ctx* ctx, int32_t* M, float* margins);
/* Logits [M][vocab] of the last pass; only recorded while bit 0 of asd_set_debug's flags is set. */
int asd_get_last_logits(asd_ctx* ctx, int32_t* M, float* logits);
/* Debug flags: bit 0 = record the logits of every pass; bit 1 = record a per-stage device timeline.
 * Two more bits exercise the error path of the bounded device waits without hanging anything.
 * ASD_DEBUG_SHORT_WAITS: every wait of the pass kernel (ring slots, grid barrier) gives up after about a
 * millisecond instead of about two seconds. ASD_DEBUG_MISSING_ARRIVAL: the grid barrier in front of the stage
 * that finishes the cosine similarities of a pass waits for one arrival more than there are CTAs, so it can only
 * end by its budget; the pass then still runs to its end, and the call that launched it returns ASD_ERR_DEVICE_TIMEOUT with the stage and the CTA in
 * asd_last_error. The error stays set (every later pass returns it too) until asd_reset. */
#define ASD_DEBUG_LOGITS 1
#define ASD_DEBUG_TRACE 2
#define ASD_DEBUG_SHORT_WAITS 4
#define ASD_DEBUG_MISSING_ARRIVAL 8
#define ASD_DEBUG_NO_TAGGED_HANDOFF 16 /* one-row passes synchronise at the grid barrier like the others (for comparison) */
int asd_set_debug(asd_ctx* ctx, int32_t flags);
/* Timeline of the last pass (bit 1 of asd_set_debug): ns_out[n_stages][12][n_ctas]. Entries 0-3 are device
 * timestamps in ns of every CTA: 0 = stage entered, 1 = inputs of the stage ready (previous stage finished on
 * all CTAs), 2 = weight streaming done, 3 = stage left. Entries 4 and 5 are SM cycles that the CTA's first
 * consumer warp spent waiting for ring slots and working on them; entries 6 and 7 are timestamps of a GEMV stage
 * after the RMSNorm statistics and after the first activation window is in shared memory. Entries 8-10 are the
 * producer's: timestamps of its first and last copy of the stage, and the SM cycles it waited for free ring
 * slots in between (one of its lanes); entry 11 is unused. Call first with ns_out = NULL for the sizes. */
int asd_get_last_trace(asd_ctx* ctx, int32_t* n_stages, int32_t* n_ctas, int64_t* ns_out);
/* K and V rows (bf16 patterns, n_kv_heads*head_dim each) of one layer (0-based) at one position. */
int asd_get_kv(asd_ctx* ctx, int32_t layer, int32_t pos, uint16_t* k, uint16_t* v);
int asd_get_positions(asd_ctx* ctx, int32_t* n_committed, int32_t* draft_cursor);
int asd_get_stats(asd_ctx* ctx, asd_stats* stats);

/* ------------------------------------------------------------------------------------------------------
 * The dense product of the prompt path on its own (kernel-level tests and micro-benchmarks; Section 3.2: the
 * prompt goes through every sublayer of M at once):  C[M, N] = A[M, K] * W[N, K]^T.
 * All pointers are DEVICE pointers, 16-byte aligned: A and W bf16 row-major (raw 16-bit patterns), K % 8 == 0;
 * C float row-major [M, N]; dev_status 8 ints that the call clears on the stream and that stay 0 unless a
 * bounded device-side wait expired (word 0 != 0: C is not valid). The kernel is enqueued on the stream; the
 * call does not wait for it. Nothing is allocated. Returns ASD_ERR_ARG for bad arguments, ASD_ERR_CUDA when
 * the tensor maps cannot be encoded or the launch fails. */
int asd_gemm_bf16(void* cuda_stream, int32_t M, int32_t N, int32_t K, const uint16_t* A, const uint16_t* W, float* C,
                  int32_t* dev_status);

/* ------------------------------------------------------------------------------------------------------
 * The sublayer building block on its own (kernel-level tests and micro-benchmarks): one fused
 *   xin = gain ? bf16(RMSNorm(x; gain, eps)) : x ;  a = W xin ;  epilogue
 * for M <= 9 rows. All pointers are DEVICE pointers.
 *   x        : gain != NULL -> float [M, n_in] ; gain == NULL -> bf16 [M, n_in]
 *   W        : bf16 [n_rows, n_in]; n_in % 8 == 0
 *   epilogue : ASD_EPI_PLAIN    out = float [M, n_rows]
 *              ASD_EPI_SWIGLU   rows of W alternate gate_i, up_i (n_rows even);
 *                               out = bf16 [M, n_rows/2] = silu(gate) * up
 *              ASD_EPI_RESIDUAL out = float [M, n_rows], updated IN PLACE: out += a (the residual add), and
 *                               cos[m] = cosine(out before, out after)  -- the summand of C_l, Section 3.2
 *   scratch  : >= asd_fused_gemv_scratch_bytes() bytes, 256-byte aligned; its first 256 bytes must be zero
 *              before the first use and are left zero by every call.
 * Errors: ARG, NOMEM (scratch too small), CUDA. Asynchronous on the stream.
 */
#define ASD_EPI_PLAIN 0
#define ASD_EPI_SWIGLU 1
#define ASD_EPI_RESIDUAL 2
size_t asd_fused_gemv_scratch_bytes(void);
int asd_fused_gemv(void* cuda_stream, int32_t M, int32_t n_in, int32_t n_rows, const void* x, const uint16_t* gain,
                   float eps, const uint16_t* W, int32_t epilogue, void* out, float* cos, void* scratch,
                   size_t scratch_bytes);

/* The same fused sublayer product for callers that must not allocate (the paper has no counterpart; this is
 * a deployment convenience). Some hosts of this library cannot call cudaMalloc at the point where they need
 * the kernel: code running inside a memory pool that owns the whole device, a plug-in whose host forbids
 * driver allocations after start-up, or a latency-critical loop in which an allocation would synchronise the
 * device. For them the cross-CTA scratch of asd_fused_gemv lives in a fixed array inside the library image
 * (about 42 KB of device memory per GPU that loads the library, held until the process exits), so the caller
 * passes only inputs and outputs. Arguments and results are exactly those of asd_fused_gemv.
 *   - Limit: the array covers launch plans of up to 296 CTAs. A shape whose plan needs more (very many rows
 *     with a long reduction dimension and many activation rows) is rejected with ASD_ERR_NOMEM and a message on
 *     stderr; use asd_fused_gemv with your own scratch for those.
 *   - The first call on each device looks up the array's device address (that device must be current) and
 *     configures the kernels; make that first call outside any stream capture. The address is kept per device
 *     ordinal for the life of the process: it does not survive a cudaDeviceReset, after which this entry point
 *     must not be used again in the same process. The set-up itself is serialised between host threads.
 *   - All calls on a device share the one array: two calls whose kernels can overlap on the GPU (different
 *     streams without ordering, or several host threads) race on it. Order them on one stream.
 *   - The call itself allocates nothing: no cudaMalloc, cudaFree or allocating library routine.
 * Errors: ARG, NOMEM (plan larger than the built-in array), CUDA. Asynchronous on the stream. */
int asd_fused_gemv_static(void* cuda_stream, int32_t M, int32_t n_in, int32_t n_rows, const void* x,
                          const uint16_t* gain, float eps, const uint16_t* W, int32_t epilogue, void* out, float* cos);

/* Algorithm 1 as a pure host function (no context): C[L] -> remove_attn[L], remove_mlp[L]. */
int asd_admg(const float* C, int32_t L, const asd_admg_params* p, uint8_t* remove_attn, uint8_t* remove_mlp);
/* Algorithm 1 plus the MLP threshold of ASD_USE_CS_MLP: C_attn[L], C_mlp[L] (C_mlp may be NULL unless that flag is
 * set) -> remove_attn[L], remove_mlp[L]. Pure host function. Errors: ARG. */
int asd_admg_ext(const float* C_attn, const float* C_mlp, int32_t L, const asd_admg_params* p, uint8_t* remove_attn,
                 uint8_t* remove_mlp);

#ifdef __cplusplus
}
#endif
#endif /* ASD_H_ */
