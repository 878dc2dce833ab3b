/*
 * aed_dec.h — C ABI of the batched autoregressive decoder for attention
 * encoder-decoder (AED) speech models on NVIDIA B200 (sm_100a).
 *
 * The paper (Section "Methods", paragraph "Transferring model capacity from
 * decoder to encoder"; abstract) identifies the autoregressive cross-attention
 * Transformer decoder as the inference bottleneck of models such as Canary-1B
 * and measures the effect of its depth (24 vs 4 layers, Table "rtfx").  This
 * library runs exactly that part: greedy decoding steps of a pre-LN Transformer
 * decoder for a batch of utterances with ragged encoder lengths (the paper's
 * two padding axes, Section "Introduction" and Figure "efficiency_cubes", are
 * both handled without padding: encoder frames are packed, and finished
 * utterances are compacted away on the device).
 *
 * One decoding step, per active utterance u with t_u tokens already consumed:
 *   x  = E[token] * sqrt(d) + PE(t_u)                      (sinusoidal positions)
 *   per layer:  x += Wo  . selfattn (LN1(x))   over the t_u+1 cached positions
 *               x += Woc . crossattn(LN2(x))   over the T_u encoder frames of u
 *               x += W2 . relu(W1 . LN3(x) + b1) + b2
 *   logits = LNf(x) . Wout^T (+ bout);   next = lowest index of the maximum
 *
 * General rules
 *   - Every pointer marked DEVICE is device memory owned by the caller and must
 *     stay valid while the handle uses it; HOST pointers are read during the
 *     call only.  The library allocates no device memory: all of its device
 *     state lives in the caller's workspace.
 *   - All work is enqueued on the stream given at creation.  Calls return once
 *     the work is enqueued, except aed_dec_greedy_decode, which synchronises
 *     the stream once before returning its status.
 *   - Utterances are addressed by their index in the batch given to
 *     aed_dec_precompute_cross_kv; compaction of finished rows is internal.
 *   - No call throws or aborts; every failure is a negative aed_status_t and
 *     leaves the decode state unchanged.  aed_dec_last_error gives the text.
 *   - Matrices are row-major [out_features, in_features].  With dtype
 *     AED_DTYPE_F32 every tensor (weights, biases, LayerNorm parameters,
 *     embedding, encoder states, K/V caches) is fp32 and all arithmetic is fp32
 *     FMA.  With AED_DTYPE_BF16 every tensor is bf16; accumulation, LayerNorm
 *     statistics, softmax and the residual stream stay fp32.
 */
#ifndef AED_DEC_H_
#define AED_DEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aed_dec aed_dec_t; /* opaque handle; host memory owned by the library */

typedef enum {
    AED_OK = 0,
    AED_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, length 0, d_model not divisible by heads ... */
    AED_ERR_CAPACITY = -2,    /* batch, frame count or step count beyond what the handle was created for */
    AED_ERR_STATE = -3,       /* call out of order, e.g. a step before any precompute */
    AED_ERR_CUDA = -4,        /* a CUDA runtime call or launch failed */
    AED_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired */
    AED_ERR_UNSUPPORTED = -6  /* shape outside what the kernels support (see aed_dec_create) */
} aed_status_t;

enum { AED_DTYPE_F32 = 0, AED_DTYPE_BF16 = 1 };
/* Storage of the cross-attention keys and values: in the configured dtype, or (bf16 configuration only) rounded to
 * the 8-bit floating-point format E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; nearest, ties to even,
 * saturating at 448).  The paper does not discuss storage formats; the store is the largest stream of a decode step
 * and the 8-bit form halves it.  Projections, softmax and accumulation are unchanged. */
enum { AED_CROSS_KV_DTYPE = 0, AED_CROSS_KV_E4M3 = 1 };

typedef struct {
    int32_t n_layers, d_model, n_heads, d_ffn, vocab, d_enc;
    int32_t dtype;                /* AED_DTYPE_F32 or AED_DTYPE_BF16 */
    int32_t max_batch;            /* most utterances in one batch */
    int32_t max_total_enc_frames; /* most encoder frames in one batch, summed over utterances */
    int32_t max_enc_len;          /* most encoder frames of one utterance */
    int32_t max_dec_len;          /* most decoding steps of one utterance */
    int32_t bos_id;               /* start token of aed_dec_greedy_decode */
    int32_t eos_id;               /* < 0: no end-of-sequence stopping */
    float ln_eps;                 /* LayerNorm epsilon (biased variance) */
    int32_t cross_kv_format;      /* AED_CROSS_KV_DTYPE or AED_CROSS_KV_E4M3 */
    void *workspace;              /* DEVICE, 256-byte aligned, at least aed_dec_workspace_bytes() */
    size_t workspace_bytes;
    void *stream;                 /* cudaStream_t of the caller (NULL = default stream) */
} aed_dec_config_t;

/* All members are DEVICE pointers to tensors of the configured dtype.  The per-layer members are HOST arrays
 * of n_layers DEVICE pointers (the arrays are copied at creation, the tensors are borrowed).  A NULL bias
 * pointer (or a NULL per-layer bias array) means "no bias".
 * w_qkv rows: d query rows, then d key rows, then d value rows.  w_kv_c rows: d key rows, then d value rows. */
typedef struct {
    const void *embed;      /* [vocab, d_model] */
    const void *final_ln_g; /* [d_model] */
    const void *final_ln_b; /* [d_model] */
    const void *w_out;      /* [vocab, d_model] */
    const void *b_out;      /* [vocab] or NULL */
    const void *const *ln1_g, *const *ln1_b;   /* [d_model] */
    const void *const *w_qkv, *const *b_qkv;   /* [3 d_model, d_model], [3 d_model] */
    const void *const *w_o, *const *b_o;       /* [d_model, d_model], [d_model] */
    const void *const *ln2_g, *const *ln2_b;   /* [d_model] */
    const void *const *w_q_c, *const *b_q_c;   /* [d_model, d_model], [d_model] */
    const void *const *w_kv_c, *const *b_kv_c; /* [2 d_model, d_enc], [2 d_model] */
    const void *const *w_o_c, *const *b_o_c;   /* [d_model, d_model], [d_model] */
    const void *const *ln3_g, *const *ln3_b;   /* [d_model] */
    const void *const *w_ff1, *const *b_ff1;   /* [d_ffn, d_model], [d_ffn] */
    const void *const *w_ff2, *const *b_ff2;   /* [d_model, d_ffn], [d_model] */
} aed_dec_weights_t;

/*
 * Bytes of device workspace a handle with this configuration needs (the workspace and stream members are
 * ignored).  Returns 0 if the configuration is invalid or unsupported.
 */
size_t aed_dec_workspace_bytes(const aed_dec_config_t *config);

/*
 * Create a decoder for one model (the decoder definition above; depth and width per the paper's Table
 * "rtfx" variants are free parameters).  Validates the configuration, carves the caller's workspace into
 * self-attention K/V caches, the cross-attention K/V store, activation buffers and decode state, and fills
 * the positional table.  Supported shapes: head_dim = d_model / n_heads == 64; d_model, d_ffn, d_enc
 * multiples of 64; vocab >= 2; cross_kv_format = AED_CROSS_KV_E4M3 only with dtype = AED_DTYPE_BF16.  Otherwise
 * AED_ERR_UNSUPPORTED.  In the bf16 configuration the call also builds, in the workspace and on the caller's stream,
 * the LayerNorm-fold constants of the folded projections and, per layer, the composite of the self-attention output
 * projection and the cross-attention query projection (a d x d matrix product per layer: creation takes milliseconds,
 * not microseconds).  On success *out receives the handle.
 */
aed_status_t aed_dec_create(const aed_dec_config_t *config, const aed_dec_weights_t *weights, aed_dec_t **out);

/*
 * Start a new batch: compute the cross-attention keys and values of every layer,
 *   Kc = X Wkc^T + bkc,  Vc = X Wvc^T + bvc,
 * once for all packed encoder frames (they depend only on the encoder output, which the paper's decoder
 * attends to at every step), and reset the decode state (t_u = 0, every utterance active).
 *   enc_packed  DEVICE [sum(enc_lens), d_enc], configured dtype, utterance after utterance, no padding
 *   enc_lens    HOST   [batch], each in 1..max_enc_len
 *   batch       1..max_batch
 */
aed_status_t aed_dec_precompute_cross_kv(aed_dec_t *dec, const void *enc_packed, const int32_t *enc_lens,
                                         int32_t batch);

/*
 * One decoding step (the per-token computation the paper names as the bottleneck) for every utterance that
 * takes part: consumes tokens_in[u] at position t_u, appends its self-attention key/value to the cache, and
 * advances t_u by one.
 *   tokens_in   DEVICE int32 [batch], indexed by utterance; entries of idle utterances are ignored
 *   active      DEVICE uint8 [batch] or NULL; an utterance takes part if it is not retired and (active == NULL
 *               or active[u] != 0).  Utterances are retired only by aed_dec_greedy_decode.
 *   logits_out  DEVICE float [batch, vocab] or NULL; rows of idle utterances are left untouched
 *   next_out    DEVICE int32 [batch] or NULL; greedy choice (lowest index on ties); idle entries untouched
 * Errors: AED_ERR_STATE before a precompute; AED_ERR_CAPACITY if a participating utterance already holds
 * max_dec_len tokens (checked on the host from the steps issued so far, so only reliable when every step uses
 * active == NULL; with masks the device also refuses to write past the cache and raises a sticky error that
 * the next aed_dec_greedy_decode or aed_dec_sync_status reports).
 */
aed_status_t aed_dec_step(aed_dec_t *dec, const int32_t *tokens_in, const uint8_t *active, float *logits_out,
                          int32_t *next_out);

/*
 * Feed a fixed-length prompt in one pass instead of prompt_len single steps (the paper's decoder is fed a
 * fixed-length task / language prompt before the transcript: caption of Fig. "tpsdist").  Every utterance of the
 * batch consumes prompt[u][0 .. prompt_len-1] at positions 0 .. prompt_len-1: one batched causal pass in which the
 * step weights are streamed once for all positions (in chunks of floor(max_batch / batch) positions, because the
 * (utterance, position) rows share the step's row buffers; size max_batch >= batch * prompt_len for a single pass).
 * The result is what prompt_len calls of aed_dec_step would leave: the self-attention caches hold prompt_len
 * positions, t_u = prompt_len, and logits_out / next_out describe the last prompt position.
 *   prompt      DEVICE int32 [batch, prompt_len], row-major by utterance
 *   logits_out  DEVICE float [batch, vocab] or NULL
 *   next_out    DEVICE int32 [batch] or NULL: greedy choice after the whole prompt
 * Must directly follow aed_dec_precompute_cross_kv (AED_ERR_STATE otherwise); continue with aed_dec_step.
 * AED_ERR_CAPACITY if prompt_len > max_dec_len; AED_ERR_UNSUPPORTED in the fp32 configuration.
 */
aed_status_t aed_dec_prefill(aed_dec_t *dec, const int32_t *prompt, int32_t prompt_len, float *logits_out,
                             int32_t *next_out);

/*
 * aed_dec_step for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * deployment aid).  Some hosts of this library run where cudaMalloc is off limits: a serving process whose
 * device memory pool was sized and frozen at start-up, a real-time thread that may not block in the driver,
 * or an embedding runtime that hands out no allocator at all.  Such a caller can still hand in buffers it already owns for inputs and
 * outputs, but has nowhere to put the flash-decoding scratch (per (row, head, 64-position chunk): running
 * max, running sum and 64 partial accumulators).  This variant keeps that scratch in a fixed array inside the
 * library image instead of the workspace region; everything else is as in aed_dec_step, with the same
 * arguments, results and errors.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   - Only the fp32 configuration splits attention into chunks and therefore uses the scratch; the bf16 step
 *     merges its chunks inside one thread block, writes no partials, and runs unchanged through this call.
 *   - The array holds aed_dec_static_scratch_bytes() = 8 MiB, and every GPU whose context loads the library
 *     keeps that much memory until the process exits.  An fp32 batch that needs more
 *     (batch x n_heads x ceil(max(max_enc_len, max_dec_len) / 64) x 264 bytes) is refused with
 *     AED_ERR_CAPACITY and nothing is launched; bf16 batches are never refused on this ground.
 *   - The first call on each device looks up the array's device address (the device of the handle's stream
 *     must be current, as for every call); make that first call outside any stream capture.
 *   - All handles and all calls on one device share the one array, and it keeps whatever the previous call
 *     left in it.  The step writes every partial before reading it, so nothing needs clearing, but two calls
 *     whose kernels overlap on the GPU (different streams, or different handles on different streams) race
 *     on it: serialise them.
 */
aed_status_t aed_dec_step_static_scratch(aed_dec_t *dec, const int32_t *tokens_in, const uint8_t *active,
                                         float *logits_out, int32_t *next_out);
size_t aed_dec_static_scratch_bytes(void);

/*
 * Greedy decoding of the whole batch from the start token: step, feed each argmax back as the next input,
 * retire an utterance once it produced max_len[u] tokens (or, when eos_id >= 0, right after it emitted eos_id),
 * compact the remaining rows on the device, and stop when none is left.  Must directly follow a precompute.
 *   max_len     HOST   [batch], each in 1..max_dec_len
 *   tokens_out  DEVICE int32 [batch, max_dec_len]; tokens_out[u][j] is the argmax after consuming j+1 inputs;
 *               entries at and beyond out_lens[u] are set to -1
 *   out_lens    DEVICE int32 [batch]
 * Synchronises the stream before returning.
 */
aed_status_t aed_dec_greedy_decode(aed_dec_t *dec, const int32_t *max_len, int32_t *tokens_out, int32_t *out_lens);

/*
 * Continuous batching: instead of one batch that thins out until its longest utterance ends, the handle keeps a fixed
 * number of slots, and a new utterance enters a slot as soon as the previous one has left it, so every step runs with
 * (nearly) all rows occupied.  The paper counts padded positions as wasted computation (Introduction; "Methods",
 * bucketing) and shows the spread of output lengths per second of audio (Fig. "tpsdist"); the tail of a static batch
 * is the decoder-side form of that waste.  An utterance's tokens do not depend on what else is in the batch.
 *
 * aed_dec_open_slots: replaces the current batch by `slots` empty slots (1..max_batch).  Slot s owns rows
 *   s * max_enc_len .. (s + 1) * max_enc_len - 1 of the cross-K/V store, so slots * max_enc_len <= max_total_enc_frames
 *   is required (AED_ERR_CAPACITY otherwise).
 * aed_dec_admit: a new utterance takes slot `slot` (empty, or left by an utterance that is finished): the cross-K/V of
 *   its frames is computed into the slot's rows (step A0 for one utterance), its position returns to 0 with the start
 *   token, and out_lens[slot] is set to 0 if out_lens is not NULL.
 *     enc      DEVICE [enc_len, d_enc] row-major, config dtype, 16-byte aligned; read during the call's kernels only
 *     enc_len  1..max_enc_len;  max_len 1..max_dec_len (forced length, an upper bound when eos_id >= 0)
 *   Without an end-of-sequence id a slot whose utterance still decodes is refused (AED_ERR_STATE); with one the
 *   caller must have seen out_lens[slot] > 0 first.
 * aed_dec_greedy_steps: up to n_steps greedy steps over the occupied slots (fewer when the host already knows that no
 *   slot decodes any more; *steps_done, if not NULL, receives the number issued).  Tokens and lengths are written as by
 *   aed_dec_greedy_decode, indexed by slot: tokens_out DEVICE int32 [slots, max_dec_len], out_lens DEVICE int32
 *   [slots]; out_lens[slot] becomes the utterance's length in the step that retires it, which is how the caller
 *   learns that the slot is free (copy its tokens out before admitting the next utterance).  Entries of tokens_out
 *   beyond an utterance's length keep whatever an earlier occupant left there.  Does not synchronise.
 * aed_dec_step, aed_dec_prefill and aed_dec_greedy_decode do not run on slots (AED_ERR_STATE); a later
 * aed_dec_precompute_cross_kv returns the handle to batch operation.
 */
aed_status_t aed_dec_open_slots(aed_dec_t *dec, int32_t slots);
aed_status_t aed_dec_admit(aed_dec_t *dec, int32_t slot, const void *enc, int32_t enc_len, int32_t max_len,
                           int32_t *out_lens);
aed_status_t aed_dec_greedy_steps(aed_dec_t *dec, int32_t n_steps, int32_t *tokens_out, int32_t *out_lens,
                                  int32_t *steps_done /* HOST out, may be NULL */);

/*
 * The whole stream through the slots: utterances enter in arrival order (order[i], or 0, 1, 2, ... if order is NULL) as
 * slots become free, and leave with their tokens.  Without an end-of-sequence id the host knows the step in which every
 * utterance ends, issues exactly the steps up to the next departure and never waits for the device; with one it issues
 * poll_steps steps at a time and reads the slots' lengths back.
 *   enc_packed  DEVICE [sum(enc_lens), d_enc], utterance i at rows off[i] .. off[i+1] (index order, not arrival order)
 *   enc_lens, max_lens, order   HOST [n]
 *   tokens_out  HOST int32 [n, max_dec_len] (pinned memory keeps the host from waiting on every departure); row i holds
 *               out_lens[i] tokens, entries beyond are unspecified
 *   out_lens    HOST int32 [n]
 *   steps_out, row_steps_out   HOST, may be NULL: steps issued, and (slot, step) pairs that held a decoding utterance
 *               by the host's bounds (their ratio over `slots` is the occupancy)
 * The slots' token rows live in the workspace.  Synchronises the stream before returning.
 */
aed_status_t aed_dec_decode_stream(aed_dec_t *dec, const void *enc_packed, const int32_t *enc_lens, const int32_t *max_lens,
                                   const int32_t *order, int32_t n, int32_t slots, int32_t poll_steps, int32_t *tokens_out,
                                   int32_t *out_lens, int64_t *steps_out, int64_t *row_steps_out);

/* Synchronise the stream and report any sticky device-side error (AED_OK if none). */
aed_status_t aed_dec_sync_status(aed_dec_t *dec);

/*
 * The status that a value of the device-side error word stands for (host-only helper, no device access; the
 * paper has no counterpart): 0 -> AED_OK, 1 (a step was asked of an utterance whose self-attention cache is
 * full) -> AED_ERR_CAPACITY, anything else (a kernel gave up a bounded wait) -> AED_ERR_TIMEOUT.
 */
aed_status_t aed_dec_status_of_error_word(int32_t error_word);

/*
 * Measurement aid (the paper has no counterpart): with profiling enabled the library records a CUDA event on
 * its stream before and after every kernel launch.  aed_dec_profile_enable synchronises the stream, switches
 * the mode and clears the record.  aed_dec_profile_read synchronises the stream and returns, per kernel family
 * that launched, its name (static string), the sum of its launch durations in milliseconds and its number of
 * launches; the return value is the number of families written (at most max_families) or a negative status.
 * Events cost a few microseconds per launch: never time a throughput figure with profiling on.
 */
aed_status_t aed_dec_profile_enable(aed_dec_t *dec, int32_t enable);
int32_t aed_dec_profile_read(aed_dec_t *dec, int32_t max_families, const char **names /* HOST out */,
                             double *ms /* HOST out */, int64_t *launches /* HOST out */);

/* Number of kernels the handle has launched so far (host-side count, for benchmarks). */
int64_t aed_dec_launch_count(const aed_dec_t *dec);

/* Free the handle's host state.  NULL is allowed.  Device memory is the caller's and is not touched. */
void aed_dec_destroy(aed_dec_t *dec);

/* Text of the last error of this handle ("" if none); valid until the next call on the handle. */
const char *aed_dec_last_error(const aed_dec_t *dec);

/* Text of the last error of a failed aed_dec_create on this thread. */
const char *aed_dec_create_error(void);

#ifdef __cplusplus
}
#endif
#endif /* AED_DEC_H_ */
