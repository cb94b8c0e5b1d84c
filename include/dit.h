/*
 * libdit — one denoising step of a Diffusion Transformer on one B200 (sm_100a).
 *
 * The paper's serving system dispatches, per scheduling round, "diffusion steps" of requests to
 * GPU workers (Section 4, request lifecycle; Section 3 problem formulation: a request has a
 * resolution and S_i strictly dependent steps, one running at a time).  This library is the
 * single-GPU step those schedules dispatch: a stack of adaLN-Zero DiT blocks run over a batch of
 * requests at mixed image resolutions, packed into one variable-length batch with block-diagonal
 * attention per request (the mechanism behind the paper's batching of small-resolution steps,
 * Section 5 "selective continuous batching", generalised to mixed lengths).
 *
 * Conventions
 *   - C ABI, no exceptions, nothing aborts or prints.  Every call returns a dit_status; on error
 *     no kernel has been launched by that call unless stated otherwise.
 *   - "device" pointers are CUDA device memory of the current device, "HOST" pointers are host
 *     memory.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Tokens, cond and weights cross the boundary as bf16; `out` is fp32.  Inside, GEMM operands
 *     are fp16 (bf16 weights ~N(0,0.02) convert exactly), accumulation, the residual stream and the
 *     modulation vectors are fp32.  Every narrowing store saturates: a value beyond fp16's range is
 *     written as +-65504, never as infinity, so one request's overflow cannot become NaN in another
 *     (masked attention probabilities are zeros multiplied by the neighbouring request's values).
 *     DIT_FLAG_BF16_OPERANDS keeps bf16 operands instead.
 *   - The caller owns every buffer, including the workspace; the context owns only what it carves
 *     from the workspace.  No entry point below allocates device memory.
 *   - A context is not thread-safe; calls on one context must be issued serially (they may be
 *     asynchronous on one stream).  Different contexts share nothing (the library keeps no state
 *     outside a context and its workspace, dit_modulation_noalloc's fixed scratch apart) and may
 *     step at the same time on different streams.
 *
 * The block (per request r, tokens x [L_r, H], cond c [C]); the paper runs such blocks through
 * PyTorch and does not restate them, so this is the standard adaLN-Zero form:
 *   m = W_ada^T SiLU(c) + b_ada, split as (shift_a, scale_a, gate_a, shift_m, scale_m, gate_m)
 *   h = LN(x) * (1 + scale_a) + shift_a            LN over H, biased variance, eps, no affine
 *   [Q|K|V] = h W_qkv + b_qkv                       head j = columns j*d..(j+1)*d-1 of each third
 *   a = concat_j softmax(Q_j K_j^T / sqrt(d)) V_j   over the L_r tokens of this request only
 *   x = x + gate_a * (a W_o + b_o)
 *   h = LN(x) * (1 + scale_m) + shift_m
 *   x = x + gate_m * (gelu_tanh(h W_1 + b_1) W_2 + b_2)
 */
#ifndef DIT_H_
#define DIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DIT_MAX_REQUESTS 64 /* upper bound on dit_config.max_requests */

typedef struct dit_ctx dit_ctx; /* opaque */

typedef enum {
  DIT_OK = 0,
  DIT_ERR_INVALID_ARG = 1,      /* NULL pointer, negative count, bad index */
  DIT_ERR_SHAPE = 2,            /* dimensions the kernels do not support, lengths that do not add up */
  DIT_ERR_CAPACITY = 3,         /* more tokens / requests / blocks than the context was sized for */
  DIT_ERR_NOT_LOADED = 4,       /* a block in [0, n_blocks) has no weights yet */
  DIT_ERR_UNSUPPORTED_ARCH = 5, /* the current device is not compute capability 10.x */
  DIT_ERR_CUDA = 6,             /* a CUDA runtime/driver call failed; see dit_last_error */
  DIT_ERR_TIMEOUT = 7,          /* a kernel gave up on a bounded wait (device status word) */
  DIT_ERR_INTERNAL = 8
} dit_status;

typedef struct {
  int32_t hidden;           /* H; multiple of 64, <= 4096 */
  int32_t n_heads;          /* nh; H = nh * head_dim */
  int32_t head_dim;         /* d; 64 or 128 */
  int32_t mlp_hidden;       /* F; multiple of 64 */
  int32_t cond_dim;         /* C; 1..4096 */
  int32_t max_blocks;       /* weight slots carved from the workspace */
  int32_t max_total_tokens; /* capacity T_max of one packed batch */
  int32_t max_requests;     /* capacity R_max, <= DIT_MAX_REQUESTS */
  float ln_eps;             /* LayerNorm epsilon (1e-6 in every benchmark configuration) */
  uint32_t flags;           /* DIT_FLAG_* bits; 0 = the plain block */
} dit_config;

/* Model-variant parts of the block, as in the FLUX / SD3 class models the paper serves (Section 6.1
 * lists them; the paper does not restate their layers).  Both act on queries and keys only, after the
 * QKV projection and before attention, and are fused into that projection's epilogue.
 *   DIT_FLAG_QK_RMSNORM  per head: q <- q / sqrt(mean(q^2) + ln_eps) * q_norm, same for k with k_norm
 *   DIT_FLAG_ROPE_2D     2-D rotary term per head: the first d/8 channels stay; the next (d - d/8)/2
 *                        turn with the token's patch row, the last (d - d/8)/2 with its patch column;
 *                        in a group of n channels, pair (2i, 2i+1) turns by p * 10000^(-2i/n).  Text
 *                        tokens sit at (0, 0).  Needs the requests' geometry: dit_step_forward_requests
 *                        or dit_denoise_step (dit_step_forward returns DIT_ERR_INVALID_ARG). */
#define DIT_FLAG_QK_RMSNORM 1u
#define DIT_FLAG_ROPE_2D 2u
/* Reduced-precision mode, off in every benchmark configuration: the four GEMMs of a block take e4m3
 * operands.  Each row of a left operand is scaled so that its largest magnitude maps to 448 and rounded
 * to e4m3: the modulated LayerNorm outputs by the LayerNorm kernel itself, the attention output and the
 * GELU output (which are produced tile by tile) by a row-quantisation pass of their own; each output
 * channel of the four weight matrices likewise at load time; the accumulator (fp32, exact products) is
 * scaled back in the epilogue.  Everything else stays as it is.  Errors grow to several per cent of the
 * output's rms; not available for two-stream blocks. */
#define DIT_FLAG_FP8_GEMM 4u
/* bf16 operands instead of fp16: the weights are kept as given (no conversion), the 16-bit
 * activations (LayerNorm outputs, q/k/v, attention probabilities and output, GELU output) are stored
 * as bf16, accumulation, residual stream and output stay fp32.  For checkpoints whose activations do
 * not fit fp16's range (the fp16 path clamps such values to +-65504 instead of overflowing, see the
 * Conventions above).  bf16 keeps 8 significant bits instead of 11, so the error against an exact
 * evaluation is several times that of the fp16 path.  Plain sequential and parallel blocks only:
 * the flag cannot be combined with the other three, and two-stream blocks are refused. */
#define DIT_FLAG_BF16_OPERANDS 8u

/* One request of the paper's problem statement (Section 3): an image resolution, a position in
 * its denoising schedule and the diffusion time of this step.  Image tokens = (height/16) *
 * (width/16) (Section 6.1: L = H*W/16^2; Table 1: 256/1024/4096/16384 for 256^2..2048^2). */
typedef struct {
  int32_t height, width;  /* pixels, positive multiples of 16 */
  int32_t n_text_tokens;  /* >= 0; appended after the image tokens of the request */
  float timestep;         /* t of this step; read by dit_timestep_cond / dit_denoise_step, else carried */
  int32_t step_index;     /* which of the request's S_i steps this is; carried for the caller */
} dit_request;

/* Device pointers, bf16, row-major [in, out] (y = x W + b).  A NULL bias means zero.
 *   w_ada [C, 6H]  b_ada [6H]   chunk order: shift_a, scale_a, gate_a, shift_m, scale_m, gate_m
 *   w_qkv [H, 3H]  b_qkv [3H]   columns: Q | K | V
 *   w_o   [H, H]   b_o   [H]
 *   w_fc1 [H, F]   b_fc1 [F]
 *   w_fc2 [F, H]   b_fc2 [H]
 *   q_norm [d]     k_norm [d]   RMS-norm scales (read with DIT_FLAG_QK_RMSNORM; NULL means ones) */
typedef struct {
  const void *w_ada, *b_ada, *w_qkv, *b_qkv, *w_o, *b_o, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
  const void *q_norm, *k_norm;
} dit_block_weights;

/* Bytes of device workspace a context of this configuration needs (0 if the configuration is
 * invalid).  Covers converted weights for max_blocks blocks, the fp32 residual stream, the
 * intermediate activations, the modulation vectors, staging for dit_step_forward_host and the
 * tensors and intermediates of the shell calls (dit_load_shell_weights and below). */
size_t dit_workspace_bytes(const dit_config *cfg);

/* Creates a context on the current device.  `workspace` is device memory, 1024-byte aligned, at
 * least dit_workspace_bytes(cfg) long; it must outlive the context.  Fails with
 * DIT_ERR_UNSUPPORTED_ARCH on anything but sm_100 (there is no fallback path). */
dit_status dit_ctx_create(const dit_config *cfg, void *workspace, size_t workspace_bytes, dit_ctx **out);
dit_status dit_ctx_destroy(dit_ctx *ctx);

/* Copies block `block_idx`'s ten tensors into the context (weights are re-laid out as fp16
 * [out, in] for the tensor-core kernels, biases widened to fp32).  Asynchronous on `stream`; the
 * caller's tensors may be freed once the stream has passed this point. */
dit_status dit_load_block_weights(dit_ctx *ctx, int32_t block_idx, const dit_block_weights *w, void *stream);

/* The parallel form of the block (the single-stream blocks of the FLUX family the paper serves):
 * one modulation triple, attention and MLP read the same modulated LayerNorm output, and one output
 * projection runs over their concatenation:
 *   (shift, scale, gate) = W_ada^T SiLU(c) + b_ada;   h = LN(x)(1 + scale) + shift
 *   a = attention(h W_qkv + b_qkv);  u = gelu_tanh(h W_fc1 + b_fc1);  x = x + gate * ([a | u] W_out + b_out)
 * Device pointers, bf16, row-major [in, out]; a NULL bias means zero, NULL q_norm / k_norm mean ones.
 *   w_ada [C, 3H]  b_ada [3H]   w_qkv [H, 3H]  b_qkv [3H]   w_fc1 [H, F]  b_fc1 [F]
 *   w_out [H + F, H] (attention rows first)  b_out [H]      q_norm [d]  k_norm [d]
 * A stack may mix both forms block by block; a block slot holds whichever form was loaded last.
 * The step runs 5 kernels for such a block instead of 7 (the attention kernel and the up-projection
 * write side by side into one [T, H + F] buffer, so the concatenation costs nothing). */
typedef struct {
  const void *w_ada, *b_ada, *w_qkv, *b_qkv, *w_fc1, *b_fc1, *w_out, *b_out, *q_norm, *k_norm;
} dit_parallel_block_weights;
dit_status dit_load_parallel_block_weights(dit_ctx *ctx, int32_t block_idx, const dit_parallel_block_weights *w,
                                           void *stream);

/* The two-stream form of the block (the double-stream / MMDiT blocks of the FLUX and SD3 families):
 * image tokens and text tokens of a request each have their own ten tensors (modulation, projections,
 * MLP, and q/k norm scales) and meet only in attention, which runs once over all tokens of the
 * request.  Such a block occupies TWO consecutive slots, block_idx (image stream) and block_idx + 1
 * (text stream); n_blocks of the step calls counts slots.  Loading either slot on its own later
 * dissolves the pair.  It needs the requests' geometry to tell image rows from text rows:
 * dit_step_forward_requests or dit_denoise_step.  Inside, every GEMM of the block visits the 256-row
 * tiles stream by stream with that stream's weights; a tile that holds rows of both streams is
 * computed once per stream and each pass stores its own rows (with the paper's token counts,
 * multiples of 256 image tokens and 512 text tokens, no tile is mixed). */
dit_status dit_load_dual_block_weights(dit_ctx *ctx, int32_t block_idx, const dit_block_weights *image_stream,
                                       const dit_block_weights *text_stream, void *stream);

/* Packer, host only, integer only (Section 6.1 token rule; requests keep their input order; inside
 * a request image tokens come first, then text tokens).  All arrays are HOST memory owned by the
 * caller: token_lens [n], cu_seqlens [n+1], row_req / row_local [sum of lens] (either may be NULL).
 * total_tokens receives the sum.  n == 0 is valid.  DIT_ERR_SHAPE for a resolution that is not a
 * positive multiple of 16 or a negative text length. */
dit_status dit_pack_requests(const dit_request *reqs, int32_t n, int32_t *token_lens, int32_t *cu_seqlens,
                             int32_t *row_req, int32_t *row_local, int32_t *total_tokens);

/* Gathers n per-request device buffers [L_r, H] bf16 (HOST array of device pointers) into one packed
 * device buffer [sum L_r, H] bf16 in request order.  Asynchronous on `stream`. */
dit_status dit_pack_tokens(dit_ctx *ctx, const void *const *per_request_tokens, const int32_t *token_lens,
                           int32_t n, void *packed_tokens, void *stream);

/* One denoising step: blocks 0..n_blocks-1 over the packed batch.
 *   packed_tokens           device [T, H] bf16, 16-byte aligned, T = sum of lens; request r owns rows
 *                           [cu[r], cu[r+1]) in input order
 *   per_request_token_lens  HOST [n_requests] int32, each >= 1; read before the call returns
 *   per_request_cond        device [n_requests, C] bf16; row r conditions request r
 *   out                     device [T, H] fp32
 * Asynchronous on `stream`; never allocates.  n_requests == 0 is a no-op.  Errors are detected on
 * the host before any launch (DIT_ERR_CAPACITY, DIT_ERR_NOT_LOADED, DIT_ERR_INVALID_ARG). */
dit_status dit_step_forward(dit_ctx *ctx, const void *packed_tokens, const int32_t *per_request_token_lens,
                            int32_t n_requests, const void *per_request_cond, int32_t n_blocks, float *out,
                            void *stream);

/* The same step with the batch described by requests (HOST array; height, width and n_text_tokens
 * are read, token lengths follow from them as in dit_pack_requests).  The only entry point of the
 * block stack that can run with DIT_FLAG_ROPE_2D, since it knows every token's patch row and column. */
dit_status dit_step_forward_requests(dit_ctx *ctx, const void *packed_tokens, const dit_request *requests,
                                     int32_t n_requests, const void *per_request_cond, int32_t n_blocks,
                                     float *out, void *stream);

/* Same step with HOST buffers: copies tokens and cond to the device, runs the step, copies `out`
 * back, and returns after everything has drained (out is valid on return).  The transfers overlap the
 * step where the data flow allows it: the tokens go in as four row slices on a copy stream of the
 * context and block 0 normalises and projects each slice as it lands; the part of the last block that
 * follows attention runs in the same row slices (only its last GEMM for parallel blocks and in the
 * e4m3 mode) and every finished slice of `out` goes back, on a stream of its own, while the next one computes.  The results are
 * those of dit_step_forward bit for bit.  Use pinned host memory (pageable memory serialises the copies). */
dit_status dit_step_forward_host(dit_ctx *ctx, const void *host_packed_tokens,
                                 const int32_t *per_request_token_lens, int32_t n_requests,
                                 const void *host_cond, int32_t n_blocks, float *host_out, void *stream);

/* The same step without the final wait, for a serving loop that keeps two steps in flight (the paper's workers
 * run step after step of their round, Section 5.2): the call returns once everything is enqueued, and
 * dit_host_wait(ctx, calls_back) blocks until the output of the latest such call (calls_back = 0) or of the one
 * before it (calls_back = 1) has arrived in its host buffer.  Successive calls on one context overlap where the
 * data allow: the tokens of call k + 1 go in as soon as block 0 of call k has read the staging buffer, and the
 * output of call k goes out while call k + 1 computes (the step itself waits for that copy before it overwrites
 * the device-side output).  Rules: issue the calls of one context on one stream; keep host_packed_tokens,
 * host_cond and host_out of a call untouched until dit_host_wait has covered it; at most two calls may be
 * outstanding (wait for call k - 1 before issuing call k + 1); an empty batch (n_requests == 0) does not count as
 * a call.  dit_step_forward_host is this call followed by dit_host_wait(ctx, 0). */
dit_status dit_step_forward_host_async(dit_ctx *ctx, const void *host_packed_tokens,
                                       const int32_t *per_request_token_lens, int32_t n_requests,
                                       const void *host_cond, int32_t n_blocks, float *host_out, void *stream);
dit_status dit_host_wait(dit_ctx *ctx, int32_t calls_back);

/* Reads (with a device synchronisation) the device status word that kernels set when a bounded wait
 * runs out; returns DIT_OK or DIT_ERR_TIMEOUT and clears the word. */
dit_status dit_ctx_poll_status(dit_ctx *ctx);

/* Test hook: device pointers to the context's intermediates of the LAST block run by the last
 * step (h = second LayerNorm+modulate output, qkv, a = attention output, u = GELU output are fp16;
 * mod [R, n_blocks, 6H] and stream [T, H] are fp32).  Valid until the next call on the context. */
typedef enum { DIT_TAP_H = 0, DIT_TAP_QKV = 1, DIT_TAP_ATTN = 2, DIT_TAP_U = 3, DIT_TAP_MOD = 4, DIT_TAP_STREAM = 5 } dit_tap;
dit_status dit_debug_tap(dit_ctx *ctx, dit_tap which, const void **ptr, int64_t *rows, int64_t *cols,
                         int32_t *elem_bytes);

/* Test hooks that stand in for a memory checker.
 * dit_debug_poison fills every activation region of the workspace (residual stream, h, qkv, a, u,
 * modulation vectors, row scales, staging buffers, shell intermediates; not the weights) with 0xFF
 * bytes, which read as NaN in every floating-point format used there, and writes a fixed pattern into
 * the 1 KiB guard areas that follow the regions.  A step run afterwards turns any read of a row it
 * never wrote into NaN in its output.  Asynchronous on `stream`.
 * dit_debug_check_guards synchronises the device, compares the guard areas with the pattern and
 * returns the number of damaged guards in *n_damaged (0 after any correct step). */
dit_status dit_debug_poison(dit_ctx *ctx, void *stream);
dit_status dit_debug_check_guards(dit_ctx *ctx, int32_t *n_damaged);

/* Measurement hook: while enabled, one thread of every attention CTA that sweeps at least 16 key blocks, and of every
 * GEMM CTA that lives 20 us or more, reads the SM's cycle counter and the global nanosecond timer at its start and end
 * and leaves cycles * 1000 / ns (the SM clock in MHz it ran at; attention also its cycles per key block) in the
 * context's status area (last writer wins).  The call synchronises the device, returns the values left since the
 * previous call (0 if none; any pointer may be NULL), clears them and sets the new state.  The step is power-capped,
 * so the clock a kernel actually runs at inside a step (which a sampler outside the process cannot attribute to a
 * kernel) is what its tensor-pipe utilisation has to be read against. */
dit_status dit_debug_clock_probe(dit_ctx *ctx, int32_t enabled, int32_t *attention_mhz, int32_t *cycles_per_key_block,
                                 int32_t *gemm_mhz);

/* Test hook for the failure path: launches one CTA that waits, with the library's bounded-wait
 * routine and a limit of about 50 microseconds, on a barrier that nothing ever signals.  The wait runs
 * out, the kernel returns normally and sets the device status word, so the next dit_ctx_poll_status
 * returns DIT_ERR_TIMEOUT (once).  Nothing hangs or faults; the context stays usable. */
dit_status dit_debug_expire_wait(dit_ctx *ctx, void *stream);

/* Per-kernel timing for benchmarks.  While enabled, every kernel launch of a step is bracketed by
 * a pair of CUDA events on the step's stream (events are created on demand and kept; no device
 * memory is allocated).  dit_ctx_read_timing synchronises the device, adds up the elapsed time and
 * the number of launches per kernel kind since the last read (HOST arrays of DIT_KERNEL_KINDS
 * entries) and starts a new accumulation. */
typedef enum {
  DIT_KERNEL_MODULATION = 0, DIT_KERNEL_LN_MODULATE = 1, DIT_KERNEL_GEMM_QKV = 2, DIT_KERNEL_ATTENTION = 3,
  DIT_KERNEL_GEMM_PROJ = 4, DIT_KERNEL_GEMM_FC1 = 5, DIT_KERNEL_GEMM_FC2 = 6,
  DIT_KERNEL_QUANTIZE = 7, /* e4m3 mode only: row quantisation of the attention and GELU outputs */
  DIT_KERNEL_KINDS = 8
} dit_kernel_kind;
dit_status dit_ctx_set_timing(dit_ctx *ctx, int32_t enabled);
dit_status dit_ctx_read_timing(dit_ctx *ctx, double *ms_by_kernel, int64_t *launches_by_kernel);

/* adaLN modulation vectors with no allocation at all (the paper has no counterpart; this exists for
 * hosts that cannot allocate device memory: a plugin called inside another runtime's execution
 * phase, a process whose memory pool belongs to a framework, a caller that was handed fixed buffers
 * and nothing else).  It needs no context and no workspace.
 *   mod_out[r, :] = W_ada^T SiLU(cond[r, :]) + b_ada        device [n_requests, 6H] fp32
 *   cond device [n_requests, C] bf16; w_ada device [C, 6H] bf16, 16-byte aligned (it is read with
 *   16-byte loads; DIT_ERR_INVALID_ARG otherwise, as for a mod_out that is not 4-byte aligned or a
 *   cond / b_ada that is not 2-byte aligned); b_ada device [6H] bf16 or NULL (zero)
 * The result is that of the `mod` vectors dit_step_forward computes for that block (the same kernel; a
 * context with many blocks may sum the cond channels in wider groups, which moves the last fp32 bits).  The fp32 copy of
 * the bias, which the context path keeps in the caller's workspace, lives here in a fixed 96 KiB
 * array inside the library image (every GPU that loads the library holds it until the process
 * exits).  Limits: hidden a multiple of 64 and <= 4096, cond_dim <= 4096, n_requests <=
 * DIT_MAX_REQUESTS; anything larger returns DIT_ERR_CAPACITY, an unsupported hidden DIT_ERR_SHAPE,
 * and nothing is launched.  The first call on a device looks the array's device address up and
 * raises the kernel's shared-memory limit; make that first call outside any stream capture.  All
 * calls share the one array, which keeps the previous call's bias until the next call rewrites
 * it (zeros for a NULL bias), so two calls whose kernels overlap on the GPU (different streams)
 * race: issue calls on one stream, or order them with events.  Asynchronous on `stream`. */
dit_status dit_modulation_noalloc(const void *cond, const void *w_ada, const void *b_ada, int32_t n_requests,
                                  int32_t cond_dim, int32_t hidden, float *mod_out, void *stream);

/* ------------------------------------------------------------------------------------------------
 * The rest of a denoising step around the block stack.  In the paper a request's latent is the only
 * state that lives from one step to the next and the only thing that moves between workers
 * (Section 4, latent transfer between rounds); a step takes the latent, runs the transformer over
 * all of its tokens (Section 2) and the sampler writes the next latent.  The paper leaves these
 * parts to the model code it serves; the forms here are the usual ones of latent DiTs:
 *
 *   latent z_r   fp32 [16, h/8, w/8]; 2 x 2 patches, flattened in (channel, dy, dx) order to 64
 *                numbers, patches in row-major (py, px) order: one token per 16 x 16 pixels
 *   tokens       image row (py, px): patch W_in + b_in + pos(py, px), rounded to bf16, where the
 *                first H/2 channels of pos encode py and the last H/2 encode px, each half being
 *                [sin(p w_k) | cos(p w_k)], w_k = 10000^(-k/(H/4)), k < H/4;
 *                text rows: taken as given (already H wide), after the image rows of the request
 *   cond         e(t) = [cos(t f_k) | sin(t f_k)], f_k = 10000^(-k/128), k < 128;
 *                c = SiLU(e W_t1 + b_t1) W_t2 + b_t2 (+ pooled), rounded to bf16
 *   final layer  (shift, scale) = SiLU(c) W_fa + b_fa;  y = LN(x)(1 + scale) + shift;
 *                v_tok = y W_out + b_out for image rows; un-patchified into v shaped like z
 *   sampler      explicit Euler step of the rectified-flow ODE: z <- z + dsigma * v,
 *                dsigma = sigma_next - sigma_cur
 *
 * Buffers that hold one array per request are concatenated in request order: `latents` and
 * `velocity` are device fp32, request r starting at element 64 * (image tokens of requests before
 * r); `text_tokens` is device bf16 [sum of n_text_tokens, H] (may be NULL when that sum is 0).
 * Requests are HOST arrays; height, width, n_text_tokens and timestep are read.  These calls need
 * hidden % 64 == 0 (as everywhere) and cond_dim % 8 == 0.  All are asynchronous on `stream`,
 * allocate nothing, and detect argument errors on the host before any launch.
 * ------------------------------------------------------------------------------------------------ */
#define DIT_LATENT_CHANNELS 16
#define DIT_PATCH_DIM 64  /* 16 channels x 2 x 2 */
#define DIT_T_EMB_DIM 256

/* Device pointers, bf16, row-major [in, out]; a NULL bias means zero.
 *   w_in [64, H]   b_in [H]      w_t1 [256, C]  b_t1 [C]     w_t2 [C, C]  b_t2 [C]
 *   w_fa [C, 2H]   b_fa [2H]  (shift | scale)   w_out [H, 64]  b_out [64] */
typedef struct {
  const void *w_in, *b_in, *w_t1, *b_t1, *w_t2, *b_t2, *w_fa, *b_fa, *w_out, *b_out;
} dit_shell_weights;

/* Copies the ten tensors into the context (W_out is re-laid out as fp16 for the tensor-core
 * kernel, biases widened to fp32).  DIT_ERR_SHAPE if cond_dim is not a multiple of 8. */
dit_status dit_load_shell_weights(dit_ctx *ctx, const dit_shell_weights *w, void *stream);

/* cond_out [n, C] bf16 (device) from the requests' timesteps; pooled is device fp32 [n, C] or NULL. */
dit_status dit_timestep_cond(dit_ctx *ctx, const dit_request *requests, int32_t n, const float *pooled,
                             void *cond_out, void *stream);

/* packed_tokens [T, H] bf16 (device), T = sum over requests of image + text tokens. */
dit_status dit_embed_latents(dit_ctx *ctx, const float *latents, const void *text_tokens,
                             const dit_request *requests, int32_t n, void *packed_tokens, void *stream);

/* x [T, H] fp32 (device, 16-byte aligned; the output of dit_step_forward), cond [n, C] bf16 (device) -> velocity. */
dit_status dit_final_layer(dit_ctx *ctx, const float *x, const dit_request *requests, int32_t n,
                           const void *cond, float *velocity, void *stream);

/* latents += dsigma[r] * velocity, request by request; dsigma is a HOST array [n]. */
dit_status dit_sampler_update(dit_ctx *ctx, float *latents, const float *velocity, const dit_request *requests,
                              int32_t n, const float *dsigma, void *stream);

/* The whole step in one call: conditioning, embedding, blocks 0..n_blocks-1, final layer and the
 * update of `latents` in place.  `velocity` (device, same layout) also receives v when not NULL.
 * Intermediates live in the context's workspace (the packed tokens share the staging buffer of
 * dit_step_forward_host).  DIT_ERR_NOT_LOADED without shell or block weights. */
dit_status dit_denoise_step(dit_ctx *ctx, float *latents, const void *text_tokens, const dit_request *requests,
                            int32_t n, const float *dsigma, const float *pooled, int32_t n_blocks,
                            float *velocity, void *stream);

/* One scheduling round on this worker, as the paper's execution model has it (Section 5.2: in a
 * round request i runs q_i consecutive steps; Section 5.3: requests of a batch leave it as they finish
 * their steps): request r runs steps_in_round[r] >= 0 steps, all requests that still have a step left
 * forming the packed batch of each step, so the batch shrinks as requests complete their quota.
 *   sigmas  HOST [n, sigma_stride] fp32: sigmas[r, k] is request r's noise level before its k-th step
 *           of this round and sigmas[r, k + 1] after it (sigma_stride >= largest step count + 1); the
 *           step's diffusion time is t = 1000 * sigma, its Euler increment sigma[k + 1] - sigma[k]
 *   latents, text_tokens, pooled: as for dit_denoise_step, for the FULL request list; latents are
 *           updated in place, those of a request with no step left stay untouched
 * Equal to calling dit_denoise_step once per step on the requests still active.  Asynchronous on
 * `stream`; a few small device-to-device copies (pooled rows) are issued when the batch shrinks. */
dit_status dit_denoise_round(dit_ctx *ctx, float *latents, const void *text_tokens, const dit_request *requests,
                             int32_t n, const int32_t *steps_in_round, const float *sigmas, int32_t sigma_stride,
                             const float *pooled, int32_t n_blocks, void *stream);

/* Number of kernel launches issued by the last dit_step_forward, dit_denoise_step or dit_denoise_round on this context. */
int64_t dit_last_launch_count(const dit_ctx *ctx);

const char *dit_status_string(dit_status s);
const char *dit_last_error(const dit_ctx *ctx); /* detail of the last failure on this context ("" if none) */

#ifdef __cplusplus
}
#endif
#endif /* DIT_H_ */
