/*
 * lasad.h -- C ABI of the B200 (sm_100a) LASAD operator library.
 *
 * LASAD = causal linear attention with Spatial-Aware Decay over a raster-flattened
 * h x w token grid (the SAD recurrence and the SAD rule of Section 3.4; Algorithm 1's
 * loop body).  Per (batch, head) a d_k x d_v state s is carried:
 *
 *     s_i = g_i * s_{i-1} + k_i v_i^T ,      o_i = scale * q_i^T s_i ,      s_{-1} = state_in
 *
 * where g_i is the head's decay constant gamma_h (data-independent decay, Section 3.3),
 * except at a row-boundary step, where it is exactly 1.  With absolute 0-based index i,
 * `prefix_len` leading non-grid tokens (a class token) and `grid_w` tokens per row,
 * step i is a boundary iff
 *
 *     grid_w > 0  and  i >= prefix_len  and  (i - prefix_len + 1) mod grid_w == 0 ,
 *
 * i.e. the step that absorbs the last token of a grid row; prefix_len = 0 is the paper's
 * rule "t mod w = 0" for 1-based t.  grid_w = 0 disables the rule (plain 1-D decay).
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned by the caller and must stay valid until the
 *     given stream has passed the call.  `lasad_params` and the ctx handle are HOST memory.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising.  lasad_create and lasad_reserve allocate device
 *     memory; lasad_forward allocates only in the case described at lasad_reserve.
 *   - Return value: LASAD_OK or a negative LASAD_ERR_*.  On an argument error nothing is
 *     launched and no output is touched.  The library never aborts the process.
 *   - Base pointers of q, k, v, o must be 16-byte aligned and every stride, in bytes, a
 *     multiple of 16; the innermost (channel) dimension is contiguous.  state is contiguous
 *     fp32 [B, H, dk, dv], 16-byte aligned.
 *   - Supported: dk == dv in {32, 64}; dtype F32 or BF16 (q, k, v, o share it; state, decay
 *     and all accumulation are fp32); any B, H, T >= 1.  Otherwise LASAD_ERR_UNSUPPORTED.
 *   - One ctx is bound to one device, which must be the current device at every call that
 *     takes the ctx (otherwise LASAD_ERR_INVALID_ARG), and may be used from one host thread at a
 *     time; its prefill calls share scratch storage (state slots, work counters), so two
 *     lasad_forward calls on one ctx must not overlap on the device (issue them on one stream,
 *     or order the streams).
 *   - A stride of 0 is accepted only for a dimension of one element.
 *   - decay (and gate) values must lie in [0, 1] and be finite: they are device data, which the
 *     library does not inspect; values outside that range give undefined results (no fault).
 */
#ifndef LASAD_H_
#define LASAD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    LASAD_OK = 0,
    LASAD_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, bad alignment or stride  */
    LASAD_ERR_UNSUPPORTED = -2, /* valid but outside the supported set above                 */
    LASAD_ERR_CUDA = -3,        /* a CUDA runtime/driver call failed (see lasad_last_cuda_error) */
    LASAD_ERR_TIMEOUT = -4      /* a bounded device-side wait expired (see lasad_last_device_status) */
};

enum { LASAD_F32 = 0, LASAD_BF16 = 1 };

/* Options for lasad_set_option. */
enum {
    LASAD_OPT_PREFILL_IMPL = 0, /* 0 auto (bf16, d = 64: 4 when B * H <= SMs / 3 and T > 1920 or
                                   B * H <= SMs / 2 and T > 3968, else 3 when B * H <= SMs / 3 and
                                   T > 128, else 5 when T > 3968 unless B * H fills whole rounds of
                                   2 * SMs to 93 % or more, else 2; other shapes 1),
                                   1 CUDA-core fp32 kernel,
                                   2 tcgen05 kernel with one CTA per (batch, head) at a time,
                                   3 tcgen05 kernel streaming (batch, head, chunk) tasks through
                                   persistent CTAs, 4 as 2 with few long sequences cut into segments
                                   that run side by side (two launches; 2 where nothing is cut),
                                   5 tcgen05 kernel with one CTA per SM whose two chunk pipelines
                                   work on one sequence at a time, the work cut evenly over the SMs */
    LASAD_OPT_PREFILL_CHUNK = 1,/* CUDA-core prefill chunk length: 0 auto, else 16/32/64          */
    LASAD_OPT_DECODE_TPU = 2,   /* decode: threads per (b,h) state; 0 auto, else 32/64/128/256 */
    LASAD_OPT_WAIT_LIMIT = 3    /* iteration cap of device-side waits; 0 = library default   */
};

typedef struct lasad_params {
    int32_t B, T, H, dk, dv; /* T = tokens in this call (ignored by lasad_decode_step)        */
    int32_t grid_w;          /* w: tokens per grid row; 0 = boundary rule off                  */
    int32_t prefix_len;      /* P: leading non-grid tokens; 0 = the paper's literal rule       */
    int32_t dtype;           /* LASAD_F32 or LASAD_BF16: element type of q, k, v, o            */
    int64_t t0;              /* absolute 0-based sequence index of the call's first token      */
    float scale;             /* multiplies o; the paper's operator has none: pass 1.0f         */
    int32_t reserved;        /* must be 0                                                      */
    /* element strides of the (batch, token, head) dimensions; channels are contiguous.
       [B,T,H,d] contiguous is {T*H*d, H*d, d}.  lasad_decode_step reads [0] and [2] only.   */
    int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];
} lasad_params;

typedef struct lasad_ctx lasad_ctx;

/* Creates a context on CUDA device `device`: a status word, work counters and the scratch storage
 * of the prefill kernels (state slots at the cuts of sequences, relay slots, per-pair flags; about
 * 60 MiB in all).  Which later calls may allocate as well is said at lasad_reserve,
 * lasad_forward_host and lasad_forward_gated; no other call allocates. */
int lasad_create(lasad_ctx** out, int device);
int lasad_destroy(lasad_ctx* ctx);
int lasad_set_option(lasad_ctx* ctx, int option, int value);

/*
 * Makes the context's relay storage large enough for prefill calls with B * H <= units.  The
 * task-streaming tensor-core prefill passes each chain's carried state (the s of the SAD
 * recurrence, Section 3.4) from the CTA that absorbed one chunk of the sequence to the CTA that
 * absorbs the next through one 32 KiB slot per (batch, head) in context-owned device memory.
 * lasad_create allocates 1024 slots.  A lasad_forward call with more (batch, head) pairs than
 * the context holds grows the storage first (cudaMalloc, which synchronises the device and must
 * not happen inside a stream capture); calling lasad_reserve up front keeps lasad_forward
 * allocation-free.  The same call sizes the 4-byte-per-pair flag array of lasad_forward_gated
 * (lasad_create provides for 65536 pairs).
 */
int lasad_reserve(lasad_ctx* ctx, int64_t units);

/*
 * Full-sequence (teacher-forced) prefill: the SAD recurrence (Section 3.4) evaluated for T
 * tokens per (batch, head) in chunk-parallel form -- intra-chunk decayed scores
 * (Q K^T o D) V plus the carried state, D built on the fly from the tokens' (row, col)
 * grid positions.
 *
 *   q, k    [B,T,H,dk]  (strided)      decay      [H] fp32, gamma_h in [0,1]
 *   v       [B,T,H,dv]                 state_in   [B,H,dk,dv] fp32 or NULL (zero state)
 *   o       [B,T,H,dv]  written        state_out  [B,H,dk,dv] fp32 or NULL; may alias state_in
 *
 * The call may be recorded into a CUDA graph (stream capture) and replayed, with one exception:
 * prefill implementation 3 numbers its launches on the host, so while `cuda_stream` is being
 * captured the default never picks it and LASAD_OPT_PREFILL_IMPL = 3 makes the call return
 * LASAD_ERR_UNSUPPORTED.
 */
int lasad_forward(lasad_ctx* ctx, const lasad_params* p,
                  const void* q, const void* k, const void* v,
                  const float* decay, const float* state_in,
                  void* o, float* state_out, void* cuda_stream);

/*
 * lasad_forward on HOST buffers: q, k, v, decay, state_in are read from, and o, state_out written
 * to, host memory (contiguous [B,T,H,d] / [H] / [B,H,dk,dv]; the strides in `p` are ignored).  Use
 * page-locked memory: the call then overlaps, one batch element at a time, the copy in of element
 * b+1, the prefill of element b and the copy out of element b-1 on two internal streams.  All
 * work is ordered after what `cuda_stream` held at the call, and `cuda_stream` is complete only
 * when o (and state_out) have arrived in host memory; the call itself does not wait.  The
 * context keeps two staging slots of one batch element each; a call that needs larger ones than
 * any before allocates them (cudaMalloc, synchronising).  Same operator, dtypes and error rules
 * as lasad_forward (Section 3.4: the SAD recurrence).
 */
int lasad_forward_host(lasad_ctx* ctx, const lasad_params* p,
                       const void* q, const void* k, const void* v,
                       const float* decay, const float* state_in,
                       void* o, float* state_out, void* cuda_stream);

/*
 * lasad_forward without a context and without any allocation.  The paper has no counterpart:
 * this exists for hosts in which this library may not allocate device memory at all -- a serving
 * process that fixes its device-memory plan at start-up and treats a later cudaMalloc as an
 * error (it synchronises the device and can fail once the plan has taken the memory), or a
 * plug-in whose host framework owns every allocation on the device.  lasad_create cannot be
 * used there, because it allocates.
 *
 * It runs the task-streaming tensor-core prefill (prefill implementation 3) on the CURRENT
 * device.  The per-(batch, head) relay slots that kernel needs live in a fixed array inside the
 * library image: 8 MiB plus a status block, held by every device that loads the library until
 * the process exits.  Limits: bf16, dk = dv = 64, B * H <= 256; anything else returns
 * LASAD_ERR_UNSUPPORTED (other argument rules as for lasad_forward).  The call makes no
 * cudaMalloc / cudaFree and calls no allocating library routine.
 *
 *   device_status   device memory, one int, or NULL.  A kernel that gives up a bounded wait
 *                   writes 1 there; the caller clears and reads it (with NULL the library's own
 *                   status block takes the write and cannot be read back).
 *
 * The first call on a device looks up the array's device address and the device's limits; make
 * that first call before starting any stream capture.  A call whose `cuda_stream` is being
 * captured returns LASAD_ERR_UNSUPPORTED and enqueues nothing: the kernel tells its calls apart by
 * a number counted on the host, which a replayed recording would repeat.  All calls on a device share the one
 * array, which keeps the previous call's contents (the library invalidates them by a call
 * counter and clears the array before the counter repeats): two calls that overlap on the GPU
 * race on it, so issue them on one stream or order the streams.  Arguments q .. state_out and
 * cuda_stream as for lasad_forward.
 */
int lasad_forward_static(const lasad_params* p,
                         const void* q, const void* k, const void* v,
                         const float* decay, const float* state_in,
                         void* o, float* state_out, int* device_status, void* cuda_stream);

/*
 * One generation step (Algorithm 1's loop body for the token at absolute index p->t0):
 * state <- g * state + k v^T in place, o = scale * q^T state, fused in one pass over the state.
 *
 *   q, k [B,H,dk], v [B,H,dv], o [B,H,dv] (strides [0] and [2] of the params)
 *   state [B,H,dk,dv] fp32, updated in place      decay [H] fp32
 */
int lasad_decode_step(lasad_ctx* ctx, const lasad_params* p,
                      const void* q, const void* k, const void* v,
                      const float* decay, float* state, void* o, void* cuda_stream);

/*
 * lasad_decode_step for sequences that are not at the same position (continuous batching, images
 * of different widths in one batch): pos [B] int32 (device) gives each sequence's absolute 0-based
 * token index, grid_w [B] int32 (device) its tokens per grid row, or NULL for p->grid_w; p->t0 is
 * ignored and the row-boundary test of the SAD rule (Section 3.4) is made per batch element on
 * the device.  Everything else as lasad_decode_step.
 */
int lasad_decode_step_pos(lasad_ctx* ctx, const lasad_params* p,
                          const void* q, const void* k, const void* v,
                          const float* decay, float* state, void* o,
                          const int32_t* pos, const int32_t* grid_w, void* cuda_stream);

/*
 * The paper's own, data-dependent form of the operator (Algorithm 1; the SAD recurrence of Section
 * 3.4 with a decay vector per token): lambda_t in [0,1]^dk, e.g. Sigmoid(Linear(x_t)), multiplies
 * the state row-wise, s_t = diag(lambda_t^spatial) s_{t-1} + k_t v_t^T, with lambda_t^spatial = 1
 * on the step that absorbs the last token of a grid row (the SAD rule) and lambda_t otherwise.
 *
 *   gate   [B,T,H,dk] (prefill) / [B,H,dk] (decode): lambda, in the dtype of q and with the
 *          strides given in k_stride.
 *   k      as in lasad_forward, or NULL: the key is tied to the gate, k_t = 1 - lambda_t (the
 *          paper's base decay, lambda_t = 1 - k_t; Algorithm 1).  k_stride always describes gate.
 *   The `decay` vector of lasad_forward has no counterpart here.  Other arguments, dtypes, sizes
 *   and error rules as for lasad_forward / lasad_decode_step.
 *
 * lasad_forward_gated with BF16 and dk == dv == 64 runs on the tensor cores (two launches: the
 * tensor-core kernel, which scales each 128-token chunk's queries and keys around a per-channel
 * reference decay and gives up a (batch, head) whose decay over one chunk falls below 2^-200 in
 * some channel, and a CUDA-core kernel that recomputes exactly the pairs given up, so every gate
 * in [0,1] is handled).  LASAD_OPT_PREFILL_IMPL picks the tensor-core kernel: 5 the balanced one
 * (one CTA per SM, as for lasad_forward), 2 the one with a CTA per (batch, head), 0 the balanced
 * one where lasad_forward's default would be 5 and the other elsewhere; 1 forces the CUDA-core
 * kernel for all pairs.
 * Other shapes and the decode step use fp32 arithmetic on CUDA cores.  The calls of one ctx
 * share a per-pair flag array: two lasad_forward_gated calls on one ctx must not overlap on the
 * device, and a call with more (batch, head) pairs than lasad_create or lasad_reserve provided
 * for (65536 by default) grows the array first, as described at lasad_reserve.
 */
int lasad_forward_gated(lasad_ctx* ctx, const lasad_params* p,
                        const void* q, const void* k, const void* v, const void* gate,
                        const float* state_in, void* o, float* state_out, void* cuda_stream);
int lasad_decode_step_gated(lasad_ctx* ctx, const lasad_params* p,
                            const void* q, const void* k, const void* v, const void* gate,
                            float* state, void* o, void* cuda_stream);

/*
 * Algorithm 1's loop body as a whole: the operator together with the element-wise steps the
 * algorithm puts around it, so that q, the gate and o each cross device memory once instead of
 * three times.  Per token (Algorithm 1, in its order):
 *
 *     q_t = SiLU(q_pre_t)            lambda_t = Sigmoid(gate_pre_t)            k_t = 1 - lambda_t  (k == NULL)
 *     s_t = diag(lambda_t^spatial) s_{t-1} + k_t v_t^T      o_t = scale * q_t^T s_t      (Section 3.4, SAD rule)
 *     out_t = Norm(o_t)
 *
 * The paper does not say which norm follows the operator; the reading taken here is a weight-free
 * RMS norm over the dv channels of each head, out = o / sqrt(mean(o^2) + norm_eps), norm_eps >= 0
 * (a learned per-channel weight, if the model has one, folds into the output projection that
 * follows).  The output projection itself and the input projections are dense matrix products and
 * are not part of these calls.
 *
 *   q_pre, gate_pre   pre-activations, with the layouts, dtypes and strides of q and gate in
 *                     lasad_forward_gated / lasad_decode_step_gated (gate_pre is described by k_stride)
 *   k                 an explicit key (then not tied to the gate), or NULL for Algorithm 1's k = 1 - lambda
 *   o                 receives the normalised output; state, state_in, state_out as in the gated calls
 *
 * Arithmetic: activations, decay products, accumulation, state and norm in fp32; with BF16 I/O
 * and dk == dv == 64 the contractions run on the tensor cores with bf16 operands, as in
 * lasad_forward_gated, and the same two-launch scheme covers every gate value.  1 - lambda is
 * formed as Sigmoid(-gate_pre), not by subtraction, so a gate close to 1 keeps its precision.
 */
int lasad_forward_fused(lasad_ctx* ctx, const lasad_params* p,
                        const void* q_pre, const void* k, const void* v, const void* gate_pre,
                        const float* state_in, void* o, float* state_out, float norm_eps,
                        void* cuda_stream);
int lasad_decode_step_fused(lasad_ctx* ctx, const lasad_params* p,
                            const void* q_pre, const void* k, const void* v, const void* gate_pre,
                            float* state, void* o, float norm_eps, void* cuda_stream);

/* After the caller has synchronised the stream: 0, or LASAD_ERR_TIMEOUT if a kernel gave up a
 * bounded wait since the last query (the flag is cleared by the query).  Synchronous copy. */
int lasad_last_device_status(lasad_ctx* ctx, int* status);

/* cudaError_t value of the last failed CUDA call on this ctx (0 if none). */
int lasad_last_cuda_error(const lasad_ctx* ctx);

/* Number of kernels this ctx has launched since creation (host-side counter). */
uint64_t lasad_launch_count(const lasad_ctx* ctx);

const char* lasad_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LASAD_H_ */
