/*
 * adit.h - C ABI of the B200 (sm_100a) batched Action Diffusion Transformer (ADiT) denoising loop.
 *
 * Operation (paper section 2.1, "Vision-Language-Action Models"; section 4.1.1, stage batching):
 * the ADiT stage of a vision-language-action model follows the VLM stage, receives each request's
 * VLM intermediate tensors (here: a per-layer key/value prefix cache, one allocation per request,
 * never packed), and runs a fixed number of diffusion steps on a batch whose size is fixed for the
 * duration of the stage, on its own CUDA stream, to produce one action chunk per request.
 *
 * The paper does not print the network's arithmetic.  This library computes, per request b:
 *
 *   x_0 = noise[b];  for k = 0..K-1:  x_{k+1} = x_k + (1/K) * v(x_k, k/K);  out[b] = x_K
 *
 * where v is a pre-norm transformer over 1 + horizon suffix tokens (one state token, then the
 * action tokens, which carry a sinusoidal time embedding through a two-layer SiLU MLP); every
 * suffix token attends, without mask or positional term, to that request's prefix keys
 * [0, prefix_len[b]) followed by all suffix keys; RMSNorm (eps inside the square root, plain gain),
 * grouped-query attention (query head h reads kv head h / (n_q_heads / n_kv_heads)), scale
 * 1/sqrt(head_dim), GeGLU MLP with tanh-approximate GELU, final RMSNorm and a linear read-out on
 * the action tokens.  dtype 1 rounds matrix-product operands to bfloat16 and accumulates in fp32;
 * the residual stream and x stay fp32.  Two variants of the model can be switched on per handle (section 2.1 leaves
 * the hand-over and the expert's attention pattern to the model): ADIT_FLAG_STATE_BLOCK_MASK and ADIT_FLAG_SUFFIX_ROPE.
 *
 * All functions return 0 (ADIT_OK) or a negative adit_status.  Nothing is enqueued when an error
 * is returned.  No function throws, aborts or synchronises the host except where stated.
 */
#ifndef ADIT_H_
#define ADIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ADIT_OK = 0,
  ADIT_E_INVALID = -1,     /* NULL pointer, B < 1, K < 1, prefix_len out of range, misaligned pointer, bad shape */
  ADIT_E_CAPACITY = -2,    /* B > max_batch, K > ADIT_MAX_STEPS */
  ADIT_E_NOT_LOADED = -3,  /* adit_denoise before a complete adit_load_weights */
  ADIT_E_UNSUPPORTED = -4, /* shape family without a compiled kernel, or a device that is not sm_100 */
  ADIT_E_CUDA = -5,        /* a CUDA runtime/driver call failed; adit_last_cuda_error() has its code */
  ADIT_E_TIMEOUT = -6      /* a bounded device-side wait ran out (reported by adit_poll_status) */
} adit_status;

#define ADIT_MAX_BATCH 64  /* upper limit of adit_config.max_batch */
#define ADIT_MAX_STEPS 64  /* upper limit of K */

#define ADIT_DTYPE_FP32 0  /* debug path: fp32 weights, prefix K/V and arithmetic */
#define ADIT_DTYPE_BF16 1  /* bf16 weights and prefix K/V, fp32 accumulation */

/* adit_config.flags */
#define ADIT_FLAG_REFERENCE_KERNELS 1 /* run the plain (non tensor-core) CUDA kernels also for bf16; debugging aid */
#define ADIT_FLAG_NO_GRAPH 2          /* enqueue kernels one by one instead of replaying a cached launch graph */
#define ADIT_FLAG_NO_PDL 4            /* no programmatic dependent launch between the loop's kernels */
#define ADIT_FLAG_MMA_SYNC_ATTENTION 8 /* attention on the legacy mma.sync path instead of tcgen05 (comparison aid) */
#define ADIT_FLAG_STATE_BLOCK_MASK 32 /* model variant: the state token attends to the prefix and itself only, not to the action tokens */
#define ADIT_FLAG_SUFFIX_ROPE 64      /* model variant: rotary embedding (pairs j, j + head_dim/2; base 10000) on the suffix queries
                                         and keys at positions prefix_len[b] + index in the suffix; prefix keys are used as given */
#define ADIT_FLAG_ONE_SM_GEMM 128     /* projections on the one-SM kernel at every batch size (comparison aid; large batches otherwise use two-SM products) */
#define ADIT_FLAG_PERSISTENT_LOOP 16  /* small batches run as one persistent kernel instead of a kernel per phase (see adit_uses_persistent_loop) */

typedef struct adit_handle adit_handle; /* opaque; owns packed weights and a workspace on one device */

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff;
  int32_t horizon, action_dim, state_dim, time_emb_dim; /* time_emb_dim even, >= 4 */
  int32_t max_batch;      /* capacity B of one call, <= ADIT_MAX_BATCH */
  int32_t max_prefix_len; /* row capacity P_cap of every prefix_kv[b] */
  int32_t dtype;          /* ADIT_DTYPE_* */
  float rms_eps;          /* e.g. 1e-6 */
  float t_min_period, t_max_period; /* e.g. 4e-3, 4.0 */
  int32_t flags;
} adit_config;

/* One named weight tensor handed to adit_load_weights.  Matrices are row-major [in, out] (y = x W). */
typedef struct {
  const char* name;   /* see adit_load_weights */
  const void* data;   /* host or device memory, per on_device */
  int32_t dtype;      /* ADIT_DTYPE_FP32 (float) or ADIT_DTYPE_BF16 (uint16 bit patterns) */
  int32_t ndim;       /* 1 or 2 */
  int64_t shape[4];
  int32_t on_device;  /* 0: data is host memory, 1: device memory on the handle's device */
} adit_tensor;

/*
 * adit_create: allocate a handle on CUDA device `device` (paper section 4.1.1: one executable per
 * stage and batch size, set up once at initialisation).  Allocates the packed-weight store and a
 * workspace sized for max_batch.  *out is written only on success.
 * Errors: INVALID (NULL, non-positive sizes, n_q_heads not a multiple of n_kv_heads, odd
 * time_emb_dim), CAPACITY (max_batch > ADIT_MAX_BATCH), UNSUPPORTED (head_dim not in {64,128,256};
 * for dtype bf16 without the reference-kernel flag: a device that is not compute capability 10.x,
 * or d_model/d_ff/head_dim not multiples of 64; ADIT_FLAG_STATE_BLOCK_MASK together with
 * ADIT_FLAG_MMA_SYNC_ATTENTION), CUDA.
 */
int adit_create(const adit_config* cfg, int device, adit_handle** out);

/*
 * adit_load_weights: copy and repack weights (section 2.1: the model is loaded once; requests are
 * stateless).  Names, with D = d_model, F = d_ff, A = action_dim, S = state_dim, Q = n_q_heads *
 * head_dim, KV = n_kv_heads * head_dim, T = time_emb_dim:
 *   action_in.w [A,D]  action_in.b [D]   state_in.w [S,D]  state_in.b [D]
 *   time_mlp.w1 [D+T,D] (rows 0..D-1 multiply the action embedding, rows D.. the time embedding)
 *   time_mlp.b1 [D]    time_mlp.w2 [D,D]  time_mlp.b2 [D]
 *   layers.<l>.norm1.g [D]  .wq [D,Q]  .wk [D,KV]  .wv [D,KV]  .wo [Q,D]
 *   layers.<l>.norm2.g [D]  .wg [D,F]  .wu [D,F]   .wd [F,D]
 *   final_norm.g [D]   action_out.w [D,A]  action_out.b [A]
 * Q/K/V columns are head-major (column = head * head_dim + i).  May be called several times with
 * subsets; the handle becomes usable once every tensor has been seen.  Tensors that feed one fused
 * matrix (norm gain with its projections) are packed when the last of them arrives.  The call
 * synchronises the device; the caller may free its copies on return.
 * Errors: INVALID (NULL, unknown name, wrong shape or dtype code), CUDA.
 */
int adit_load_weights(adit_handle* h, const adit_tensor* tensors, int n_tensors);

/*
 * adit_denoise: enqueue the whole K-step denoising loop for B requests on `stream` (section 2.1:
 * fixed number of diffusion steps; section 4.1.1: fixed batch, own stream, per-request VLM tensors).
 *
 *   prefix_kv   HOST array of B DEVICE pointers.  prefix_kv[b] is laid out
 *               [n_layers][2 (K then V)][n_kv_heads][max_prefix_len][head_dim], element type per
 *               cfg.dtype, 16-byte aligned.  Rows >= prefix_len[b] may hold anything (NaN
 *               included) and never influence the result.  Keys are used as given.
 *   prefix_len  HOST array of B lengths, 0 <= prefix_len[b] <= max_prefix_len.
 *   state       DEVICE [B, state_dim] fp32.
 *   noise       DEVICE [B, horizon, action_dim] fp32 (x_0).
 *   K           number of Euler steps, 1..ADIT_MAX_STEPS.
 *   sm_budget   <= 0 or >= the device's SM count: use all SMs; otherwise the loop's kernels run
 *               with at most sm_budget thread blocks of one block per SM (section 4.1.2: the two
 *               stages share the GPU by SM partition).
 *   stream      a cudaStream_t (NULL = the legacy default stream).
 *   out_actions DEVICE [B, horizon, action_dim] fp32; may alias noise.
 *
 * The first call with a new (B, K, sm_budget) records the loop's kernel sequence into a CUDA graph
 * (section 4.1.1 replays one graph per stage and batch size) and keeps it in the handle; later
 * calls enqueue one small kernel that carries the per-call pointers plus one graph launch.
 *
 * Asynchronous: returns after enqueueing.  Both host arrays are consumed before it returns; the
 * device buffers must stay valid until the stream reaches the end of the call.  The result for
 * request b depends only on the weights, prefix_kv[b][.., 0:prefix_len[b], ..], state[b], noise[b]
 * and K.  It is bitwise reproducible and bitwise independent of the slot, the other requests, the
 * contents of padding rows and sm_budget; the batch size B changes how reductions are split, hence
 * the result by rounding order only.
 * A handle serves one call at a time (calls on one stream are ordered; do not share a handle
 * between streams without synchronising); two handles on two streams may overlap.
 * Stream capture (section 4.1.1: the stage as a graph per batch size): the call may be recorded into the caller's
 * own CUDA graph - it then enqueues only kernels, straight into that graph - provided a call with the same K
 * was made on this handle before, outside any capture (the time-embedding vectors are computed when K changes);
 * otherwise it returns ADIT_E_UNSUPPORTED and records nothing.  A replay uses the pointers and prefix lengths given at capture time.
 * Errors: INVALID, CAPACITY, NOT_LOADED, UNSUPPORTED (see above), CUDA.
 */
int adit_denoise(adit_handle* h, int B, const void* const* prefix_kv, const int32_t* prefix_len,
                 const float* state, const float* noise, int K, int sm_budget, void* stream,
                 float* out_actions);

/*
 * adit_denoise_host: the same call for HOST buffers (state, noise, out_actions in host memory,
 * pinned for best speed): copies the inputs to the device on `stream`, runs adit_denoise, copies the
 * result back and synchronises `stream`.  prefix_kv still holds device pointers: the prefix cache is
 * produced on the device by the VLM stage (section 4.1.2: handed over in a device buffer).
 */
int adit_denoise_host(adit_handle* h, int B, const void* const* prefix_kv, const int32_t* prefix_len,
                      const float* state_host, const float* noise_host, int K, int sm_budget,
                      void* stream, float* out_actions_host);

/*
 * Hidden-state hand-over (section 2.1: the VLM creates "hidden states or a small KV cache" for the
 * ADiT).  Where the VLM hands over hidden states, the expert projects them to the per-layer prefix
 * keys and values itself, once per call (they do not depend on the diffusion step), and the loop then
 * runs on that cache as usual:
 *   K_l = H Wk_l,  V_l = H Wv_l   for every layer l, H = hidden[b] [prefix_len[b], Dh]
 * (no normalisation, bias or rotation here: H is used as handed over).
 *
 * adit_load_prefix_projection: the 2 * n_layers matrices, all in one call, named
 *   layers.<l>.prefix_wk [Dh, KV]   layers.<l>.prefix_wv [Dh, KV]
 * with one hidden width Dh (a multiple of 64) and KV = n_kv_heads * head_dim, columns head-major as for
 * wk / wv.  Independent of adit_load_weights; a second call replaces the matrices.  Synchronises the
 * device.  Errors: INVALID (NULL, a name missing or repeated, shapes), UNSUPPORTED (fp32 handles,
 * ADIT_FLAG_REFERENCE_KERNELS, or together with ADIT_FLAG_SUFFIX_ROPE), CUDA.
 *
 * adit_project_prefix: enqueue the projection for B requests on `stream`.
 *   hidden         HOST array of B DEVICE pointers, hidden[b] = [prefix_len[b], Dh] bf16, row-major,
 *                  16-byte aligned (may be NULL where prefix_len[b] == 0)
 *   prefix_len     HOST array of B lengths, 0 <= prefix_len[b] <= max_prefix_len
 *   prefix_kv_out  HOST array of B DEVICE pointers to caches in adit_denoise's layout
 *                  [n_layers][2][n_kv_heads][max_prefix_len][head_dim] bf16; rows < prefix_len[b] are
 *                  written, rows beyond are left as they are (adit_denoise never reads them)
 *   sm_budget      as in adit_denoise
 * One tensor-core product per request (fp32 accumulation, results rounded to bf16); a request's
 * cache depends on its own hidden states and length only.  Asynchronous; both host arrays are consumed
 * before it returns.  Errors: INVALID, CAPACITY (B > max_batch), NOT_LOADED (no projection loaded), CUDA.
 */
int adit_load_prefix_projection(adit_handle* h, const adit_tensor* tensors, int n_tensors);
int adit_project_prefix(adit_handle* h, int B, const void* const* hidden, const int32_t* prefix_len,
                        void* const* prefix_kv_out, int sm_budget, void* stream);

/* adit_destroy: synchronise the device and free everything the handle owns.  NULL is accepted. */
int adit_destroy(adit_handle* h);

/* adit_poll_status: non-blocking read of the device-written status word: ADIT_OK or ADIT_E_TIMEOUT. */
int adit_poll_status(adit_handle* h);

/* adit_last_cuda_error: the cudaError_t / CUresult of the most recent ADIT_E_CUDA on this handle (0 if none). */
int adit_last_cuda_error(adit_handle* h);

/* adit_kernel_launches: number of kernels the library has launched on this handle since creation. */
int64_t adit_kernel_launches(adit_handle* h);

/*
 * adit_profile_*: optional per-launch device timing by kernel class (measurement aid; the paper's
 * serving engine profiles stage executions on the device the same way, section 4.1.2).  While
 * enabled, adit_denoise brackets every kernel launch with a pair of CUDA events on the call's
 * stream (which serialises launches that would otherwise overlap).  adit_profile_read synchronises
 * the device, adds up the elapsed milliseconds and launch counts per class into the two arrays of
 * ADIT_N_KERNEL_CLASSES entries, and clears the record.  adit_profile_class_name(i) names class i.
 */
#define ADIT_N_KERNEL_CLASSES 11
int adit_profile_enable(adit_handle* h, int on);
int adit_profile_read(adit_handle* h, double* total_ms, int64_t* launches);
const char* adit_profile_class_name(int cls);

/*
 * adit_trace_*: optional timeline of one call (measurement aid; no counterpart in the paper).  While
 * enabled, every block of the projection, attention and merge kernels stores its start time, the time its wait
 * for the preceding kernel ended, the time its main loop finished (projection: last accumulator
 * complete; attention: last key block done) and its end time (%globaltimer, ns); this works inside the replayed launch graph, so kernel overlap and gaps are seen
 * as they occur.  adit_trace_enable synchronises the device and drops the cached launch graphs.
 * adit_trace_read synchronises and writes, for the launches of the most recent call in order, ten
 * int64 each: kernel class, grid size, earliest and latest block start, earliest and latest block end,
 * earliest and latest time at which a block's wait for the preceding kernel was released, earliest and
 * latest time at which a block's main loop finished (0 where not recorded).
 * Returns the number of launches written or a negative status.
 */
int adit_trace_enable(adit_handle* h, int on);
int64_t adit_trace_read(adit_handle* h, int64_t* records, int64_t max_records);

/*
 * adit_clear_status: synchronise the device and reset the status word to ADIT_OK (after an ADIT_E_TIMEOUT has
 * been read with adit_poll_status; the handle stays usable).
 */
int adit_clear_status(adit_handle* h);

/*
 * adit_uses_persistent_loop: the number of thread blocks the single persistent kernel would use for a call
 * with B requests and this sm_budget, or 0 when such a call takes the kernel-per-phase path (host only).
 * Small batches (at most 64 suffix tokens in total, at most 4 requests) of bf16 handles run the whole loop as one
 * resident kernel of 8-block clusters (section 4.1.1: the stage as one executable on its stream; section 4.1.2: on
 * its share of the SMs): floor(sm_budget / 8) clusters, at most what the device keeps resident.  Results of the
 * two paths differ by rounding order only; within a path they do not depend on B, slot or sm_budget.
 */
int adit_uses_persistent_loop(adit_handle* h, int B, int sm_budget);

/*
 * adit_debug_wait_limit: test aid for the bounded device-side waits of the persistent kernel (no counterpart in
 * the paper).  Sets the limit of every wait to limit_ms milliseconds (default 2000) and, with withhold_level in
 * 0..7 (embed-in, embed-out, qkv, attention, o, gate/up, down, read-out), makes one block withhold its
 * completion signal of the first such level of the call, so that the waits for it run out: the kernel then returns normally,
 * adit_poll_status reports ADIT_E_TIMEOUT and the call's output is unspecified.  -1 withholds nothing.
 */
int adit_debug_wait_limit(adit_handle* h, int limit_ms, int withhold_level);

/*
 * adit_loop_trace_read: timeline of the most recent persistent-kernel call made while adit_trace_enable was on
 * (measurement aid).  Per level of the call, in order, eleven int64: level type (as in adit_debug_wait_limit),
 * blocks that took part, the earliest time a block saw the level's dependency satisfied, and the latest time over
 * the blocks of eight events (%globaltimer, ns; 0 where not recorded): dependency seen; accumulator complete
 * (projection) or key loop complete (attention); partial sums sent; partial sums received; epilogue stored;
 * level's flag published; first activation tile landed; last product issued.
 * Returns the number of levels written or a negative status.
 */
int64_t adit_loop_trace_read(adit_handle* h, int64_t* records, int64_t max_records);

/* adit_strerror: static string for a status code. */
const char* adit_strerror(int code);

/*
 * adit_debug_copy: synchronise the device and copy a named workspace buffer to host memory (test
 * aid).  Names: "x" fp32 [B*horizon, A]; "h" fp32 [B*(1+horizon), D]; "rstd" fp32 [rows];
 * "qkv", "att", "mlp", "hb" in the compute dtype.  Copies min(nbytes, buffer size) bytes and returns
 * the number copied, or a negative status.
 */
int64_t adit_debug_copy(adit_handle* h, const char* name, void* host_dst, size_t nbytes);

/*
 * adit_debug_gemm_timeout: failure-path test aid for the kernel-per-phase path.  Runs a small projection
 * in which one thread block is denied one operand copy, so that one of its bounded device-side waits
 * expires (about two seconds, the kernels' limit), the block records ADIT_E_TIMEOUT in the status word,
 * waits for its copies in flight, frees its tensor memory and returns; then runs the same projection
 * untouched.  *first_status = the status word after the first run (ADIT_E_TIMEOUT expected); returns the
 * status after the second run (ADIT_OK expected) or a host-side error.  No trap, no fault, no unbounded
 * wait.  Synchronises the stream.  The paper has no counterpart.
 */
int adit_debug_gemm_timeout(int device, int* first_status, void* stream);

/*
 * adit_debug_gemm: run the tensor-core projection kernel on its own (test aid): out[n_tok, n_feat]
 * (fp32, device) = A[n_tok, k] W[n_feat, k]^T with bf16 device operands, k a multiple of 64;
 * splits = 0 lets the library choose the k-split, 1..8 caps it, 100 * t + c (t >= 1) additionally fixes the
 * number of token tiles at t (for sweeps of the tiling; a combination the kernel has no room for falls back to
 * the nearest admissible one), splits = -2 selects the two-SM kernel (pairs of
 * thread blocks, 256 features x tile_tokens per pair), sm_budget as in adit_denoise.  Synchronises the
 * stream.  Returns a negative status, or a positive plan code splits * 1e6 + tile_tokens * 1e3 +
 * pipeline stages (splits reads 9 for the two-SM kernel).  The paper has no counterpart.
 */
int adit_debug_gemm(int device, int n_tok, int n_feat, int k, const void* a_bf16, const void* w_bf16,
                    float* out_f32, int splits, int sm_budget, void* stream);

/*
 * adit_debug_attention: run the loop's ragged-prefix attention kernels on their own (test aid; the
 * operation is the attention step of the ADiT stage, section 2.1: every suffix token attends to the
 * request's cached prefix keys/values followed by the suffix keys/values).
 *   qkv        DEVICE bf16 [B * n_tokens, (n_q_heads + 2 * n_kv_heads) * head_dim]: per token the query
 *              heads, then the key heads, then the value heads (head-major)
 *   prefix_kv, prefix_len, p_cap, layer   as in adit_denoise (prefix_kv[b] is indexed with `layer`)
 *   splits     number of key splits (1..32); with more than one, partial results go through a scratch
 *              buffer that this call allocates with cudaMalloc and frees before returning
 *   out_att    DEVICE bf16 [B * n_tokens, n_q_heads * head_dim]
 * Synchronises `stream`.  Errors: INVALID (also: qkv or out_att not 16-byte aligned), CAPACITY (B > ADIT_MAX_BATCH),
 * UNSUPPORTED (head_dim), CUDA, TIMEOUT (a bounded device-side wait ran out; the output is unspecified).
 */
int adit_debug_attention(int device, int B, int n_tokens, int n_q_heads, int n_kv_heads, int head_dim, int p_cap,
                         int layer, const void* qkv, const void* const* prefix_kv, const int32_t* prefix_len,
                         int splits, void* out_att, void* stream);

/*
 * adit_attention_static: adit_debug_attention for callers that cannot allocate device memory.  (The
 * paper has no counterpart; this entry point exists for integration, not for the method.)
 *
 * Some hosts of this library run where cudaMalloc is off limits: inside a region that a larger
 * application is recording into a CUDA graph or replaying under a memory plan fixed in advance, in a
 * real-time control loop that may not take the allocator's locks, or in a process whose device memory
 * was handed out completely at start-up.  For them the scratch that the key-split attention needs
 * (partial outputs and softmax statistics per split, plus the device copy of the prefix table) is a
 * fixed array inside the library: ADIT_STATIC_SCRATCH_BYTES = 8 MiB (+ one table) per GPU, held by
 * every GPU that loads the library until the process exits.  The call allocates and frees nothing,
 * neither through CUDA nor through any library.
 *
 * Arguments and result are those of adit_debug_attention, except:
 *   - asynchronous: the kernels are enqueued on `stream` and the call returns; nothing is synchronised;
 *   - ADIT_E_CAPACITY if splits * B * n_tokens * n_q_heads * (head_dim + 2) * 4 bytes exceed
 *     ADIT_STATIC_SCRATCH_BYTES (with splits == 1 no scratch is needed and any size is accepted);
 *   - device must be in 0..63.
 * The first call on each device looks up the array's device address (and sets the kernels' shared-
 * memory attribute); make that first call outside any stream capture.  All calls on a device share
 * the one array: it keeps whatever the previous call left (nothing in it needs clearing - each call
 * writes every partial it later reads), and two calls whose kernels overlap on the GPU (different
 * streams, no dependency) race on it.  Order such calls yourself.
 * A bounded device-side wait that runs out cannot be reported by this asynchronous call: the kernels record it in
 * a status word inside the array (cleared at the start of every call); adit_attention_static_status(device)
 * copies it out (a blocking copy, so it also waits for earlier work on the device) and returns ADIT_OK or
 * ADIT_E_TIMEOUT for the most recent call.
 */
#define ADIT_STATIC_SCRATCH_BYTES (8u << 20)
int adit_attention_static(int device, int B, int n_tokens, int n_q_heads, int n_kv_heads, int head_dim, int p_cap,
                          int layer, const void* qkv, const void* const* prefix_kv, const int32_t* prefix_len,
                          int splits, void* out_att, void* stream);
int adit_attention_static_status(int device);

/*
 * adit_debug_gemm_stamps: phase timing of the projection and attention kernels (test aid; no
 * counterpart in the paper).  Called with host_dst == NULL it arms adit_debug_gemm and
 * adit_debug_attention to record, per thread block, sixteen uint64 (%globaltimer stamps of the
 * block's phases - start, set-up done, first and last k-block landed, accumulator complete, parked,
 * sent, received, summed, epilogue done, teardown, TMEM freed - and two clock64 readings); called with
 * a host buffer of n_blocks * 16 uint64 (n_blocks <= 1024) it copies the stamps of the last such call out; with
 * host_dst == NULL and n_blocks < 0 it disarms and frees the buffer.  The buffer belongs to the device that was
 * current when it was armed; only calls on that device whose grid fits it (1024 blocks, attention 512) are
 * instrumented, all others run the plain kernels.  adit_debug_stamps_selected states that rule (host only).
 */
int adit_debug_gemm_stamps(unsigned long long* host_dst, int n_blocks);
int adit_debug_stamps_selected(int armed_device, int device, int grid_blocks, int is_attention);

/*
 * adit_debug_plan: the tiling the library would choose for a projection of n_tok tokens, n_feat output
 * features (per matrix when `dual`, a gate/up pair) and inner size k on a device with sm_count SMs
 * (host-only: needs no GPU; test aid, no counterpart in the paper).  Writes twelve int32 to out:
 * token tile width, token tiles, feature tiles, k-split (= cluster size), pipeline stages, k-blocks of 64,
 * accumulator buffers, issuing threads, tensor-memory columns, dynamic shared memory in bytes, ring bytes,
 * estimated duration in nanoseconds.  Returns ADIT_OK or ADIT_E_INVALID.
 */
int adit_debug_plan(int n_tok, int n_feat, int k, int dual, int sm_count, int32_t* out);

/*
 * adit_debug_plan_projection: as adit_debug_plan, but the plan a projection of the loop actually runs with: when
 * `allow_pair` is non-zero (the default of the loop; ADIT_FLAG_ONE_SM_GEMM clears it) large gate/up pairs go to
 * the kernel that runs one tile on a pair of SMs.  Writes thirteen int32: the twelve of adit_debug_plan, then 1 if
 * the two-SM kernel was chosen (the tile then spans 256 features on two blocks, each of which brings in half of the
 * token tile), else 0.  Host-only; returns ADIT_OK or ADIT_E_INVALID.
 */
int adit_debug_plan_projection(int n_tok, int n_feat, int k, int dual, int sm_count, int allow_pair, int32_t* out);

/*
 * adit_debug_stream_read: measurement aid (no counterpart in the paper).  Allocates `bytes` of device memory
 * (larger than the L2 cache to measure HBM), reads it `iters` times with one thread block of 512 threads on each
 * of `sm_count` SMs using 16-byte loads, and writes the achieved read bandwidth in GB/s: the memory roofline
 * that applies to a run restricted to that many SMs.  Synchronises the device.
 */
int adit_debug_stream_read(int device, size_t bytes, int sm_count, int iters, double* gb_per_s);

/*
 * adit_green_stream_*: a stream whose kernels the driver confines to a partition of at least
 * `sm_count` SMs (a green context; section 4.1.2 restricts the VLM stage's stream this way, in
 * multiples of 8 SMs).  The alternative to the sm_budget argument, which caps the grids of this
 * library's own persistent kernels: a green stream also confines kernels that were not written for a
 * budget.  create returns UNSUPPORTED where the driver has no green contexts and CAPACITY when the
 * device has fewer SMs; handle gives the cudaStream_t, sm_count the size of the partition the
 * driver granted (rounded up to its granularity).  destroy synchronises the stream first.  Nothing
 * outlives the process, and the rest of the device keeps running on all SMs.
 */
typedef struct adit_green_stream adit_green_stream;
int adit_green_stream_create(int device, int sm_count, adit_green_stream** out);
void* adit_green_stream_handle(adit_green_stream* g);
int adit_green_stream_sm_count(adit_green_stream* g);
int adit_green_stream_destroy(adit_green_stream* g);

/*
 * adit_bg_gemm_*: a looping bf16 GEMM C[m,n] = A[m,k] B[n,k]^T on a capped number of SMs, the
 * stand-in for the VLM stage that shares the GPU with the ADiT stream (section 4.1.2: the VLM
 * stream is restricted to a number of SMs so that the ADiT kernels always find free ones).
 * create allocates the operands (deterministic fill); launch enqueues `iters` repetitions on
 * `stream` using at most `sm_count` SMs (<= 0: all).  create_kind chooses the kernel: 0 = the one-SM
 * projection kernel (what create uses), 1 = the two-SM kernel (pairs of thread blocks).
 */
typedef struct adit_bg_gemm adit_bg_gemm;
int adit_bg_gemm_create(int device, int m, int n, int k, adit_bg_gemm** out);
int adit_bg_gemm_create_kind(int device, int m, int n, int k, int kind, adit_bg_gemm** out);
int adit_bg_gemm_launch(adit_bg_gemm* g, int iters, int sm_count, void* stream);
int adit_bg_gemm_destroy(adit_bg_gemm* g);

#ifdef __cplusplus
}
#endif
#endif /* ADIT_H_ */
