/*
 * jot.h -- C ABI of the JoT denoising-step library for NVIDIA B200 (sm_100a).
 *
 * JoT ("Just on Time") is token-level early stopping for masked diffusion language models.  One
 * denoising step is: a bidirectional transformer forward over the canvas (prompt followed by the
 * generation region), the vocabulary-wide LM head reduced on the fly to per-position softmax
 * statistics, the spatially adaptive acceptance test, and the in-place freeze/unmask update of
 * the canvas.  Algorithm 1 of the paper is the loop around that step.
 *
 * Conventions for every entry point
 *   - returns JOT_OK (0) or a negative jot_status; never throws, aborts or prints.
 *   - "device" pointers are CUDA global-memory addresses on the current device, "host" pointers
 *     are ordinary process memory.  Nothing is allocated on the device by the library except
 *     where stated: the caller owns weights, workspace, inputs and outputs.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it; entry points that return host values synchronise that stream themselves.
 *   - matrices are row-major; bf16 means the 16-bit brain-float storage format.
 *   - all sequences of a batch have the same canvas length L (no padding, no ragged batches).
 */
#ifndef JOT_H_
#define JOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    JOT_OK = 0,
    JOT_ERR_ARG = -1,        /* null pointer, negative size, inconsistent ranges              */
    JOT_ERR_SHAPE = -2,      /* geometry the kernels do not support (see each function)       */
    JOT_ERR_WORKSPACE = -3,  /* workspace missing, misaligned or smaller than required        */
    JOT_ERR_CUDA = -4,       /* a CUDA runtime/driver call failed: see jot_last_cuda_error()  */
    JOT_ERR_TIMEOUT = -5,    /* a bounded device-side wait expired; outputs are undefined     */
    JOT_ERR_DEVICE = -6,     /* not an sm_100 device, or the driver lacks tensor-map support  */
    JOT_ERR_LIMIT = -7       /* larger than the built-in scratch of jot_gemm_bf16_noalloc     */
} jot_status;

/* Static message for a status code. */
const char* jot_status_string(int status);
/* The cudaError_t (as int) behind the most recent JOT_ERR_CUDA on this thread, else 0. */
int jot_last_cuda_error(void);

/* Acceptance parameters: tau_max, tau_min, gamma, D of Algorithm 1 and epsilon of Eq. 4.
 * Paper defaults (Table 1 caption; Section 4.2): (90, 1, 0.5, 8) for Dream, (30, 1, 0.5, 8) for
 * LLaDA, eps = 1e-12.  1 <= D <= 32, 0 < gamma < 1 is what Eq. 5 assumes; gamma is not checked.
 * schedule_after_exit = 0: the transfer schedule ranks all masked candidates and is OR-ed with the
 * early-exit mask (Section 4.2 "Implementation details"); 1: it ranks only what early exit left.
 * gate: JOT_GATE_RATIO is the paper's test r >= tau (Eq. 8).  JOT_GATE_MAXPROB replaces it by the fixed
 * probability gate the paper contrasts JoT with (Section 2): p1 >= prob_threshold, no spatial modulation;
 * the transfer schedule and the OR are unchanged.  0 < prob_threshold <= 1 is required then.
 * JOT_GATE_GLOBAL_GAP is the global early-commit rule the paper contrasts JoT with (Section 2: once the top-2
 * confidence gap exceeds a threshold, all remaining masked positions are finalised simultaneously), read as:
 * the mean over the sequence's candidates (masked positions of the current block) of the top-2 logit gap
 * top1 - top2 is compared with gap_threshold (inclusive, in fp32) and either every candidate exits or none
 * does; schedule and OR unchanged.  The compared system stages three thresholds over decoding progress
 * (7.5 / 5.0 / 2.5, Section 6.1 "Experimental Setup"): here the threshold is one input, which a caller stepping through
 * jot_denoise_step / jot_accept_freeze may change from step to step.  Any other gate value is refused
 * (JOT_ERR_ARG).
 * schedule: how many positions the transfer schedule reveals per step inside jot_generate.  The paper leaves it
 * to "the model's default unmasking schedule" (Section 4.2, "Interaction with transfer schedules").
 * JOT_SCHEDULE_FIXED: block_len positions spread evenly over the block's steps, the remainder on the earliest
 * steps.  JOT_SCHEDULE_FRACTIONAL: ceil(positions still masked in the block / steps the block has left), the
 * adaptive rule of samplers that reveal a fraction of what remains; without early exits both give the same
 * counts.  jot_accept_freeze takes its count as an argument and ignores the field (it must still be 0 or 1). */
typedef struct {
    float tau_max, tau_min, gamma;
    int32_t D;
    float eps;
    int32_t schedule_after_exit;
    int32_t gate;            /* 0 = JOT_GATE_RATIO, 1 = JOT_GATE_MAXPROB, 2 = JOT_GATE_GLOBAL_GAP */
    float prob_threshold;    /* JOT_GATE_MAXPROB: finalise when p1 >= prob_threshold */
    float gap_threshold;     /* JOT_GATE_GLOBAL_GAP: finalise every candidate when their mean top-2 logit gap >= this */
    int32_t schedule;        /* 0 = JOT_SCHEDULE_FIXED, 1 = JOT_SCHEDULE_FRACTIONAL (jot_generate only) */
} jot_params;
enum { JOT_GATE_RATIO = 0, JOT_GATE_MAXPROB = 1, JOT_GATE_GLOBAL_GAP = 2 };
enum { JOT_SCHEDULE_FIXED = 0, JOT_SCHEDULE_FRACTIONAL = 1 };

/* Geometry of the denoiser f_theta (Algorithm 1 treats it as given).  Llama-style: RMSNorm,
 * rotate-half RoPE on absolute canvas positions, grouped-query attention without any mask, SwiGLU
 * MLP, untied LM head, no biases.  Supported: head_dim 64 or 128; d_model, d_ff and
 * n_q_heads*head_dim multiples of 64; vocab a multiple of 8; n_q_heads a multiple of n_kv_heads. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab, mask_id;
    float rope_theta, rms_eps;
} jot_model_config;

/* bf16 device pointers, BORROWED for the model's lifetime and never written.
 *   embed [vocab, d]; lm_head [vocab, d]; final_norm [d]
 *   per layer l (arrays of n_layers host-resident pointers):
 *     attn_norm[l] [d]; wqkv[l] [(nq + 2 nkv) * hd, d] (Q rows, K rows, V rows);
 *     wo[l] [d, nq * hd]; mlp_norm[l] [d]; w_gate_up[l] [2 * d_ff, d] (gate rows, then up rows);
 *     w_down[l] [d, d_ff].  Every pointer 16-byte aligned. */
typedef struct {
    const void* embed;
    const void* lm_head;
    const void* final_norm;
    const void* const* attn_norm;
    const void* const* wqkv;
    const void* const* wo;
    const void* const* mlp_norm;
    const void* const* w_gate_up;
    const void* const* w_down;
} jot_weights;

/* Generation settings of Algorithm 1.  gen_len = number of masked positions appended to the prompt;
 * steps = T; block_len = semi-autoregressive block size (gen_len for a single block; must divide
 * gen_len, and gen_len/block_len must divide steps).  exclude_mask_token != 0 keeps the mask token
 * out of the candidate predictions.  compact_finished: the paper decodes one sequence at a time, where
 * early stopping ends the loop; in a batch the loop runs until the slowest sequence is done, and with this
 * flag the forward pass only covers the sequences still decoding (same tokens and step counts, fewer rows).
 * kv_cache: the composition with a block-wise KV cache that Section 6.2 ("Composability with KV-cache
 * acceleration") measures; see jot_denoise_step_cached for what a step then computes.  All sequences work on
 * the same block and move on together once none of them has a masked position left in it (a sequence that
 * is done with the block idles, its step count stands still); compact_finished and use_cuda_graph are
 * ignored; the host reads the outcome of every step before it enqueues the next.
 * use_cuda_graph: the kernels of one step are captured on `stream` (which therefore must not already be
 * capturing) and replayed as one graph launch per step; pays off when a step is a few dozen short kernels. */
typedef struct {
    int32_t gen_len, steps, block_len;
    int32_t exclude_mask_token;
    int32_t compact_finished;   /* != 0: sequences that have finished drop out of later forward passes */
    int32_t use_cuda_graph;     /* != 0: a step is captured into a CUDA graph once and replayed */
    float temperature;          /* > 0: finalised positions receive a sample from softmax(l / temperature) */
    uint32_t seed_lo, seed_hi;  /* the 64-bit seed of jot_sampling; a row's step is its sequence's own count of
                                   denoising steps so far, so a draw does not depend on the rest of the batch */
    int32_t kv_cache;           /* != 0: decode under the block-wise KV cache (needs jot_attach_kv_cache) */
} jot_gen_config;

/* Sampling-based finalisation (Section 4.1, "Early-Exit Decision": the finalised token may be drawn from
 * the predicted distribution instead of taken as its argmax).  temperature > 0 turns it on: next to the
 * statistics, every active row also yields one draw from softmax(logits / temperature), made by the
 * Gumbel-max identity argmax_v(l_v / T - ln(-ln u_v)) inside the LM-head epilogue.  u_v = (k + 0.5) / 2^23
 * with k the top 23 bits of output number v + 1 of the splitmix64 stream whose start state is
 * mix64(seed ^ (step << 40) ^ flat_position), flat_position = b * L + i, so a draw depends only on
 * (seed, step, position, token) and can be reproduced anywhere.  The acceptance decisions still use the
 * un-tempered logits; pass the sampled array instead of the argmax array to jot_accept_freeze. */
typedef struct {
    float temperature;   /* <= 0: off */
    uint64_t seed;
    int32_t step;        /* index of this forward pass (0-based) */
} jot_sampling;

typedef struct jot_model jot_model; /* opaque; host-side object owned by the library */

/* Bytes of device workspace a model needs for batches up to max_batch sequences of canvas length up
 * to max_seq.  Returns 0 on invalid arguments. */
size_t jot_workspace_bytes(const jot_model_config* cfg, int max_batch, int max_seq);

/* Create a model over borrowed weights and a caller-owned workspace (device, 1024-byte aligned, at
 * least jot_workspace_bytes()).  Writes tables into the workspace (synchronous).  The workspace must
 * stay alive and untouched by the caller until jot_free_model.  One model must not be used from two
 * streams at once. */
int jot_init_model(const jot_model_config* cfg, const jot_weights* weights, int max_batch, int max_seq,
                   void* d_workspace, size_t workspace_bytes, jot_model** out);
int jot_free_model(jot_model* m);

/* The LM head gives every block of 128 active rows a CTA (256 rows a CTA pair) of its own, so one call can
 * take at most jot_max_active_rows(number of SMs) = 128 * (SMs rounded down to even) active rows: the masked
 * positions inside [blk_lo, blk_hi) summed over the batch, bounded by B * (blk_hi - blk_lo), which is what the
 * entry points check (JOT_ERR_SHAPE beyond it; 18,944 on a 148-SM device).  jot_lm_head_partition reports how
 * the head's schedule cuts `active_rows` rows and `vocab_tiles` vocabulary tiles over `n_ctas` CTAs (pair_mode:
 * CTA pairs): row blocks and vocabulary chunks per row block.  Host arithmetic only; exported so that the
 * schedule can be checked without a device (n_chunks >= 1 for every accepted row count). */
int jot_max_active_rows(int n_sms);
int jot_lm_head_partition(int active_rows, int n_ctas, int vocab_tiles, int pair_mode, int* n_row_blocks,
                          int* n_chunks);

/* Algorithm 1, "Compute logits" through "Compute confidence", for one step: the transformer forward
 * over d_tokens [B, L] (int32, read-only), then the LM head over the rows that are masked
 * (== mask_id) inside [blk_lo, blk_hi), reduced on the fly; logits are never stored.
 * Outputs are device arrays indexed [B, L]; only entries of active rows are written:
 *   top1_logit = largest logit, argmax = its token id (lowest id on ties), top2_logit = second
 *   largest logit (equal to top1 on an exact tie), sumexp = sum_v exp(logit_v - top1_logit),
 * so p1 = 1/sumexp and p2 = exp(top2 - top1)/sumexp (Section 4.1, "Confidence Metric").
 * d_bump_id / d_bump_val ([B, L] int32 / float, both or neither NULL) add bump_val[b,i] to the logit
 * of token bump_id[b,i] at position (b,i): a synthetic-workload hook.
 * exclude_mask_token != 0 removes column mask_id from every statistic. */
int jot_denoise_step(jot_model* m, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi,
                     int exclude_mask_token, const int32_t* d_bump_id, const float* d_bump_val,
                     float* d_top1_logit, float* d_top2_logit, float* d_sumexp, int32_t* d_argmax,
                     const jot_sampling* sampling /* nullable */, int32_t* d_sampled /* [B, L], with sampling */,
                     void* stream);

/* The single-step entry points (jot_denoise_step, jot_denoise_step_cached, jot_lm_head_stats) end, by default,
 * with a 4-byte device-to-host copy of the model's status word and a synchronisation of `stream`, so that an
 * expired device-side wait (JOT_ERR_TIMEOUT) or a token id outside [0, vocab) in d_tokens (JOT_ERR_ARG; such a
 * row is embedded as token 0, nothing is read out of bounds) comes back as their return value.
 * jot_set_sync(m, 0) turns that off: the calls return as soon as their kernels are enqueued, and the caller
 * asks for the status when it wants to (jot_read_status: synchronises `stream`, returns the same codes, and
 * clears a bad-token report so that the caller can go on with corrected input).  jot_set_sync(m, 1) restores
 * the default.  jot_generate always reads the status itself. */
int jot_set_sync(jot_model* m, int sync);
int jot_read_status(jot_model* m, void* stream);

/* Block-wise KV cache (Section 6.2, "Composability with KV-cache acceleration": JoT run inside a decoder that
 * caches keys and values block by block).  The paper names that decoder without defining it; the scheme
 * built here is the published one with a cache on both sides of the block:
 *   refresh != 0  the whole canvas goes through the network exactly as in jot_denoise_step, and every
 *                 layer's rotated keys and its values, for all L positions, stay in the attached cache;
 *   refresh == 0  only rows [blk_lo, blk_hi) go through the network; in every layer their fresh keys and
 *                 values replace the cache's entries for those positions and their queries attend over
 *                 all L positions, the others as cached.  Needs an earlier refresh with the same B and L
 *                 (else JOT_ERR_ARG).  Per step this costs (blk_hi - blk_lo) / L of the full pass's
 *                 projections; its statistics are approximate wherever the canvas has changed outside
 *                 the block since the refresh.
 * The cache is caller-owned device memory of jot_kv_cache_bytes(cfg, max_batch, max_seq) bytes, 1 KiB
 * aligned, attached with jot_attach_kv_cache (d_cache = NULL detaches) and borrowed until detached or the
 * model is freed; attaching invalidates what was cached.  Outputs and options as in jot_denoise_step. */
size_t jot_kv_cache_bytes(const jot_model_config* cfg, int max_batch, int max_seq);
int jot_attach_kv_cache(jot_model* m, void* d_cache, size_t bytes);
int jot_denoise_step_cached(jot_model* m, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi,
                            int refresh, int exclude_mask_token, const int32_t* d_bump_id,
                            const float* d_bump_val, float* d_top1_logit, float* d_top2_logit, float* d_sumexp,
                            int32_t* d_argmax, const jot_sampling* sampling, int32_t* d_sampled, void* stream);

/* The LM head + statistics part of jot_denoise_step alone, on caller-supplied final hidden states
 * d_hidden [B*L, d] bf16 (already normalised).  Uses only lm_head, vocab, mask_id and d_model of
 * the model.  Same outputs and options as jot_denoise_step. */
int jot_lm_head_stats(jot_model* m, const void* d_hidden, const int32_t* d_tokens, int B, int L,
                      int blk_lo, int blk_hi, int exclude_mask_token, const int32_t* d_bump_id,
                      const float* d_bump_val, float* d_top1_logit, float* d_top2_logit,
                      float* d_sumexp, int32_t* d_argmax, const jot_sampling* sampling, int32_t* d_sampled,
                      void* stream);

/* The same over a slice [v_lo, v_hi) of the vocabulary: top1 / argmax / top2 / sumexp of every active row taken
 * over the token ids of the slice only (argmax is a global token id; the mask token and the bump apply when they
 * fall inside the slice; sumexp is relative to the slice's own top1).  This is one rank's share of a
 * vocabulary-parallel head: statistics of disjoint slices combine exactly (top1, top2, argmax) and to fp32
 * rounding (sumexp) with jot_merge_stats, which applies to [n] arrays the associative rule the head itself uses
 * for its vocabulary chunks: top1 = max, top2 = max of the two runner-ups and the smaller top1, sumexp rescaled
 * to the new top1, argmax of the larger top1 (lower token id when equal).  Outputs may alias the first input.
 * 0 <= v_lo < v_hi <= vocab; sampling is refused on a proper slice (a draw needs the whole vocabulary).  A slice
 * that holds nothing but the excluded mask token yields top1 = -inf, sumexp = 0, argmax = INT32_MAX, the
 * neutral element of the merge. */
int jot_lm_head_stats_slice(jot_model* m, const void* d_hidden, const int32_t* d_tokens, int B, int L,
                            int blk_lo, int blk_hi, int exclude_mask_token, const int32_t* d_bump_id,
                            const float* d_bump_val, int v_lo, int v_hi, float* d_top1_logit,
                            float* d_top2_logit, float* d_sumexp, int32_t* d_argmax,
                            const jot_sampling* sampling, int32_t* d_sampled, void* stream);
int jot_merge_stats(int n, const float* a_top1, const float* a_top2, const float* a_sumexp,
                    const int32_t* a_argmax, const float* b_top1, const float* b_top2, const float* b_sumexp,
                    const int32_t* b_argmax, float* o_top1, float* o_top2, float* o_sumexp, int32_t* o_argmax,
                    void* stream);

/* Section 4.1 Eq. 4-8 and the state update of Algorithm 1 for one step, in place on d_tokens [B, L].
 * Candidates are the positions of [blk_lo, blk_hi) that hold mask_id.  For each: confidence ratio
 * r = p1/(p2 + eps) from the statistics (Eq. 4), spatial weight over the whole canvas (Eq. 5,
 * resolved = any position not holding mask_id, window radius D, positions outside the canvas
 * contribute nothing), softening (Eq. 6), threshold (Eq. 7), test r >= tau in fp32 (Eq. 8).  The
 * k_transfer candidates with the largest p1 (ties to the lower position) are chosen by the transfer
 * schedule; a candidate chosen by either rule receives its argmax.  All decisions use the canvas as
 * it was on entry.  params (host): one struct applied to all sequences, or, with per_seq_params != 0,
 * B structs, one per sequence; those travel as kernel arguments, so B <= 64 then (JOT_ERR_SHAPE beyond:
 * sequences are independent, call once per 64).
 * Outputs (device): d_n_masked [B] = candidates still masked after the update; optional
 * d_exit_reason [B, L] uint8 (bit 0 early exit, bit 1 schedule; written for finalised positions
 * only) and d_exit_step [B, L] int16 (= step_index, same positions). */
int jot_accept_freeze(const jot_params* params, int per_seq_params, int32_t mask_id, int32_t* d_tokens,
                      int B, int L, int blk_lo, int blk_hi, int k_transfer, const float* d_top1_logit,
                      const float* d_top2_logit, const float* d_sumexp, const int32_t* d_argmax,
                      int32_t* d_n_masked, uint8_t* d_exit_reason, int16_t* d_exit_step,
                      int step_index, void* stream);

/* Algorithm 1 for a batch of B independent sequences with prompts d_prompt [B, P] (int32, must not
 * contain mask_id; ids must lie in [0, vocab), else JOT_ERR_ARG).  Each sequence keeps its own block pointer and step counter and idles once
 * finished; the loop ends when no sequence has a masked position left, or after `steps` iterations.
 * Outputs: d_out_tokens [B, P + gen_len] (device); h_steps_used [B] (host) = denoising steps each
 * sequence actually ran (step speed-up = steps / steps_used, Section 6.1 "Experimental Setup"); optional
 * h_forward_passes (host, one int) = batched forward passes executed.
 * d_bump_id / d_bump_val: as in jot_denoise_step, indexed [B, P + gen_len], fixed across steps.
 * trace (nullable, any member nullable): what the paper's analysis plots are made of.  Device arrays,
 * zeroed by the call and then written by the acceptance kernel:
 *   d_exit_step [B, P + gen_len] int16: the sequence's own 1-based denoising step that finalised the
 *     position (0: prompt); d_exit_reason, same shape, uint8: bit 0 early exit (Eq. 8), bit 1 transfer
 *     schedule, both when both chose it;
 *   d_mean_ratio [steps, B] float: mean confidence ratio r (Eq. 4) over the candidates the sequence had at
 *     its s-th step (row s, 0-based; Appendix "Confidence Dynamics"); d_n_candidates, same shape, int32:
 *     how many candidates that was.  Rows past a sequence's last step stay zero.
 * Synchronises `stream` once per step to read the loop condition. */
typedef struct {
    int16_t* d_exit_step;
    uint8_t* d_exit_reason;
    float* d_mean_ratio;
    int32_t* d_n_candidates;
} jot_trace;
int jot_generate(jot_model* m, const jot_params* params, int per_seq_params, const jot_gen_config* gen,
                 const int32_t* d_prompt, int B, int P, const int32_t* d_bump_id, const float* d_bump_val,
                 int32_t* d_out_tokens, int32_t* h_steps_used, int32_t* h_forward_passes, const jot_trace* trace,
                 void* stream);

/* C[M, N] (bf16) = A[M, K] (bf16) . W[N, K]^T (bf16) with fp32 accumulation on the tensor cores,
 * optionally + residual[M, N] (bf16, may alias C).  The projection every layer of the forward is made
 * of, exported for testing and benchmarking.  K and N multiples of 8; pointers 16-byte aligned.
 * d_scratch (device, optional, 16-byte aligned, scratch_bytes long): fp32 space for split-K partial
 * sums, used when the output has too few tiles to fill the GPU and up to 4 * M * N * 4 bytes fit;
 * NULL keeps K in one piece.
 * d_status: device int32 the kernel sets non-zero if a bounded wait expires (may be NULL). */
int jot_gemm_bf16(const void* d_A, const void* d_W, const void* d_residual, void* d_C, int M, int N, int K,
                  void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream);

/* jot_gemm_bf16 for callers that must not allocate device memory.  (The paper has no counterpart
 * to this function; it exists for the library's users.)  Some code that wants this projection runs
 * where cudaMalloc is off limits: inside a latency-critical serving loop whose memory was carved up at
 * start-up, under a framework whose caching allocator must stay the only owner of the device heap, or
 * in a plugin that is handed buffers and forbidden to create its own.  jot_gemm_bf16 makes such a
 * caller bring scratch for the split-K partial sums; this variant brings its own: a fixed array of
 * JOT_NOALLOC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the library
 * holds that much memory until the process exits.  Arguments and result are those of jot_gemm_bf16
 * without the scratch pair; inputs and outputs are still the caller's.
 *   - Limit: 4 * M * N * sizeof(float) must fit in the array (M * N <= 1,048,576), else JOT_ERR_LIMIT
 *     and nothing is launched.
 *   - The first call on each device looks up the array's device address (a host-side query, no
 *     allocation); make that first call outside any stream capture.
 *   - No cudaMalloc/cudaFree and no allocating library routine is called, on any call.
 *   - All calls share the one array and it keeps whatever the previous call left there.  Nothing in it
 *     needs to start at zero: every partial sum the reduction reads is written earlier in the same
 *     call.  Two calls whose kernels overlap on the GPU (different streams, or different host threads
 *     on different streams) race on it; issue them on one stream or serialise them yourself. */
#define JOT_NOALLOC_SCRATCH_BYTES (16u << 20)
int jot_gemm_bf16_noalloc(const void* d_A, const void* d_W, const void* d_residual, void* d_C, int M, int N, int K,
                          int32_t* d_status, void* stream);

/* Optional timing of the kernels a model launches, by class, with CUDA events recorded on the launching
 * stream around each launch.  jot_profile(m, 1) starts (and clears) the accumulation, jot_profile(m, 0)
 * stops it; jot_profile_read waits for the recorded events and returns, per class, the accumulated
 * device milliseconds and the number of timed spans (host arrays of at least JOT_PROF_CLASSES entries).
 * Classes time single kernels except ROWS (active-row list + final norm / gather, two kernels). */
enum {
    JOT_PROF_EMBED = 0, JOT_PROF_RMSNORM, JOT_PROF_GEMM_QKV, JOT_PROF_ROPE, JOT_PROF_ATTENTION, JOT_PROF_GEMM_O,
    JOT_PROF_GEMM_GATE_UP, JOT_PROF_GEMM_DOWN, JOT_PROF_ROWS, JOT_PROF_LM_HEAD, JOT_PROF_MERGE, JOT_PROF_ACCEPT,
    JOT_PROF_CLASSES
};
int jot_profile(jot_model* m, int enable);
int jot_profile_read(jot_model* m, double* ms, int64_t* launches, int n_classes);

/* Failure-path self test.  Every device-side wait in this library is bounded in wall time and, on expiry,
 * makes the kernel unwind and set a status word instead of hanging.  This launches a one-CTA kernel that waits
 * (for at most limit_ns nanoseconds, <= 5e9) on a barrier nothing ever signals and writes 1 to *d_status when
 * the wait gives up, 0 if it did not.  The kernel ends normally and the context stays usable. */
int jot_selftest_wait_expiry(int32_t* d_status, uint64_t limit_ns, void* stream);

/* Number of kernels this library has launched from the calling process so far. */
int64_t jot_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* JOT_H_ */
