/*
 * eco.h -- C-ABI of the B200 (sm_100a) ECO optimizer-step library.
 *
 * ECO (arXiv 2601.22101) trains with quantized weights and NO master weights:
 * each step dequantizes the stored weight, applies the optimizer update,
 * requantizes, and injects the quantization error into the momentum buffer
 * (Algorithm 1 = OPTIM_STEP followed by ECO_QUANTIZE; Algorithm 2 for momentum
 * SGD, Algorithm 3 for Adam; quantizer and rounding of Sec. 3.1).
 *
 * All pointers named "device" are CUDA device pointers of the device the
 * context was created on; the caller owns every buffer and the stream.  The
 * library owns only its descriptor tables and a few bytes of reduction
 * scratch per tensor.  No call in this header synchronizes the device unless
 * it says so.  There is no CPU fallback: without a CUDA device every call
 * that needs one returns ECO_ERR_CUDA.
 */
#ifndef ECO_H_
#define ECO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eco_ctx eco_ctx;
typedef struct eco_host_ctx eco_host_ctx;

typedef enum eco_status {
    ECO_OK = 0,
    ECO_ERR_INVALID_ARG = 1, /* a value outside the domain of the method (see eco_step) */
    ECO_ERR_UNSUPPORTED = 2, /* a combination this build has no kernel for */
    ECO_ERR_ALIGNMENT = 3,   /* a buffer is not 16-byte aligned */
    ECO_ERR_CUDA = 4,        /* a CUDA runtime call failed; eco_last_error has its text */
    ECO_ERR_NOMEM = 5,
    ECO_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (see eco_check) */
} eco_status;

/* Weight format (Sec. 3.1; rho = largest representable magnitude). */
enum { ECO_FORMAT_FP8_E4M3 = 0, /* OCP E4M3 "FN": bias 7, rho = 448, S.1111.111 = NaN is never written;
                                   one byte per element */
       ECO_FORMAT_INT4 = 1,     /* integers -7..7, rho = 7, two's-complement nibbles, two per byte,
                                   element 2k in the low nibble; -8 is never written */
       ECO_FORMAT_FP8_E5M2 = 4 };/* OCP E5M2: bias 15, rho = 57344, infinities and NaNs are never written; one byte per
                                   element.  Not used by the paper; offered because Sec. 3.1 holds for any format
                                   with a largest magnitude rho */
/* Scale granularity (Sec. 3.1, "granularity").  Tensors are row-major [rows, cols]. */
enum { ECO_SCALE_PER_TENSOR = 0, /* 1 scale                                              */
       ECO_SCALE_PER_ROW = 1,    /* rows scales                                          */
       ECO_SCALE_PER_BLOCK = 2 };/* rows * ceil(cols / block) scales, blocks of `block`
                                    consecutive elements of one row; the last block of a
                                    row may be short                                     */
/* Stored type of a scale.  F32: s = max|x| / rho.  BF16: that quotient rounded to bf16 (nearest even); the rounded
 * value defines the grid.  E8M0: one byte b, s = 2^(b - 127), the smallest power of two with s * rho >= max|x|
 * (so nothing overflows, as with s = max|x| / rho); b = 255 is never written, an all-zero block stores b = 127.
 * The paper names power-of-two shared scales only by citation (Sec. 3.1, group-wise schemes); with block = 32 this is
 * the layout of the microscaling formats. */
enum { ECO_SCALE_F32 = 0, ECO_SCALE_BF16 = 1, ECO_SCALE_E8M0 = 2 };
enum { ECO_OPT_SGDM = 0,  /* dampened momentum SGD: m~ = beta m + (1-beta) g, theta~ = theta^ - eta m~ (Eq. 2-3) */
       ECO_OPT_ADAM = 1 };/* Adam in the form of Sec. 3.2, "Adam"                                                */
enum { ECO_ROUND_NEAREST = 0,    /* ties to the even code                                                        */
       ECO_ROUND_STOCHASTIC = 1 };/* upper neighbour with probability (x - lower)/gap; Philox4x32-10 keyed by
                                     seed, counter = (element index / 4, tensor_id, step), word = index mod 4;
                                     the top 24 bits of the word are compared with the fraction                  */
enum { ECO_INJECT_NONE = 0, /* naive master-weight removal (Sec. 3.4): the error is dropped */
       ECO_INJECT_ECO = 1,  /* the paper's method: m^ = m~ + alpha e                        */
       ECO_INJECT_EXACT = 2 };/* Appendix A: m <- m~ + e_t / eta - e_{t+1} / (eta beta) with the STORED error of the
                               previous step; reproduces master-weight momentum SGD exactly, at the price of an FP32
                               error buffer per parameter (eco_attach_error_buffers); momentum SGD only            */

typedef struct eco_config {
    int32_t format;      /* ECO_FORMAT_*                                  */
    int32_t granularity; /* ECO_SCALE_PER_*                               */
    int32_t block;       /* block length for ECO_SCALE_PER_BLOCK: 128 or 32 */
    int32_t scale_dtype; /* ECO_SCALE_F32, ECO_SCALE_BF16 or ECO_SCALE_E8M0 */
    int32_t optimizer;   /* ECO_OPT_*                                     */
    int32_t rounding;    /* ECO_ROUND_*                                   */
    int32_t injection;   /* ECO_INJECT_*; ECO_INJECT_ECO is the method    */
    int32_t reserved;    /* must be 0                                     */
} eco_config;

/* One parameter tensor and its optimizer state.  All buffers are device
 * memory, 16-byte aligned, contiguous, and must not overlap one another. */
typedef struct eco_tensor {
    void* w;           /* in/out: codes; rows*cols bytes (FP8) or rows*cols/2 bytes (INT4)        */
    void* scale;       /* in/out: scales, layout given by granularity, dtype by scale_dtype       */
    const void* grad;  /* in: gradient, bf16 [rows*cols]; re-read at every eco_step                */
    float* m;          /* in/out: first moment / momentum, f32 [rows*cols]                         */
    float* v;          /* in/out: second moment, f32 [rows*cols]; must be NULL for ECO_OPT_SGDM    */
    int64_t rows, cols;
    uint32_t tensor_id;/* selects the tensor's random stream; unique within a context              */
    uint32_t row_offset;/* 0 for a whole tensor.  For a shard made of rows [row_offset, row_offset + rows) of a
                          larger tensor: the random stream is then drawn for the elements' positions in the
                          whole tensor, so that shards round exactly like the unsplit tensor.  row_offset * cols
                          must be a multiple of 4                                                          */
} eco_tensor;

/*
 * eco_create -- bind a list of tensors that share one configuration.
 * Operation: prepares Algorithm 1 for the tensor list (host-side only apart
 * from one upload of the descriptor table).
 *   out      host; receives the context.
 *   cfg      host; copied.
 *   tensors  host array of n entries; copied (the device buffers they name are
 *            NOT copied and must outlive the context).
 *   device   CUDA device ordinal; made current for the calling thread.
 * Errors: ECO_ERR_INVALID_ARG (NULL, n == 0, rows/cols < 1, rows*cols >= 2^34,
 * INT4 with odd cols, duplicate tensor_id, v not matching the optimizer,
 * overlapping buffers, non-device pointers), ECO_ERR_UNSUPPORTED (a block other
 * than 128 or 32, unknown enum), ECO_ERR_ALIGNMENT, ECO_ERR_CUDA, ECO_ERR_NOMEM.  On error *out
 * is NULL and eco_last_error(NULL) describes the failure.  Allocates device
 * memory (tables and scratch); synchronizes the device once.
 */
eco_status eco_create(eco_ctx** out, const eco_config* cfg, const eco_tensor* tensors, size_t n, int device);

/*
 * eco_step -- one quantized training step t on every tensor of the context
 * (Algorithm 1): for each element
 *   theta^ = value(code) * scale                         (Sec. 3.1)
 *   SGDM:  m~ = beta1 m + (1-beta1) g ; theta~ = theta^ - lr m~          (Eq. 2-3)
 *   Adam:  m~, v~ updated with g ; theta~ = theta^ - lr (m~/(1-beta1^t)) / (sqrt(v~/(1-beta2^t)) + eps)
 *   scale' = max|theta~| / rho over the element's scale block ; code' = round(theta~ / scale')
 *   e = theta~ - value(code') * scale'                   (Algorithm 2/3, line 2)
 *   SGDM:  m = m~ + (1/lr)(1 - 1/beta1) e                (Algorithm 2, line 5)
 *   Adam:  m = m~ + ((1-beta1^t)/lr)(1 - 1/beta1)(sqrt(v~/(1-beta2^t)) + eps) e ; v = v~   (Algorithm 3, line 5)
 * and writes code', scale', m, v in place.  No full-precision weight is ever stored.
 *   step   t >= 1, the 1-based count of updates including this one.
 *   seed   key of the stochastic-rounding stream (ignored for ECO_ROUND_NEAREST).
 *   beta2, eps are ignored for ECO_OPT_SGDM.
 *   cuda_stream  a cudaStream_t (NULL = the legacy default stream).
 * Asynchronous: enqueues its kernels on cuda_stream and returns; it never
 * synchronizes and never allocates.  Consecutive steps of one context must be
 * ordered on the device (same stream, or events), because they share the
 * context's reduction scratch.  The call can be recorded by a stream capture
 * (CUDA graph); a replay repeats the recorded step index, seed and
 * hyper-parameters.  With ECO_SCALE_PER_TENSOR the reduction scratch alternates
 * between two halves from one call to the next (each call clears the half the
 * next one accumulates into), so a graph for that granularity must hold an even
 * number of consecutive eco_step calls.
 * Errors: ECO_ERR_INVALID_ARG for lr <= 0 or non-finite (alpha = (1/lr)(..) is
 * undefined, Eq. 7), beta1 outside (0,1) (1/beta1), Adam beta2 outside (0,1),
 * eps < 0, step < 1; ECO_ERR_CUDA for a failed launch.  On ECO_ERR_INVALID_ARG
 * nothing is launched and no buffer is modified.
 */
eco_status eco_step(eco_ctx* ctx, float lr, float beta1, float beta2, float eps,
                    uint64_t step, uint64_t seed, void* cuda_stream);

/*
 * eco_step_ex -- eco_step with the two additions the paper's training recipe makes to OPTIM_STEP
 * (Sec. 4.2: AdamW with weight decay 0.1, gradient clipping at norm 1; Algorithms 1-3 leave both
 * inside the optimizer's step function):
 *   grad_scale    every gradient element is multiplied by this factor first (the clipping factor
 *                 min(1, c / ||g||), or 1 / loss-scale; the caller computes it).  1 = off.
 *   weight_decay  decoupled decay lambda: theta^ <- theta^ - (lr lambda) theta^ before the update,
 *                 for SGDM and Adam alike.  0 = off.
 * The error injection is unchanged.  With grad_scale = 1 and weight_decay = 0 the call is eco_step.
 * Errors: as eco_step, plus ECO_ERR_INVALID_ARG for a NULL or non-zero-reserved struct, a negative
 * or non-finite weight_decay, or a non-finite grad_scale.
 */
typedef struct eco_hyper {
    float lr, beta1, beta2, eps;
    float weight_decay, grad_scale;
    uint64_t step; /* 1-based */
    uint64_t seed;
    uint64_t reserved; /* must be 0 */
} eco_hyper;
eco_status eco_step_ex(eco_ctx* ctx, const eco_hyper* hyper, void* cuda_stream);

/*
 * eco_step_begin / eco_amax_buffer / eco_step_end -- eco_step_ex cut in two at the one point where a
 * per-tensor scale needs the whole tensor (Sec. 3.1: s = max|x| / rho over everything that shares the
 * scale), for tensors whose rows are split across several GPUs:
 *   eco_step_begin   pass 1 on every tensor of the context: max |theta~| into the context's amax vector.
 *   eco_amax_buffer  device pointer and length of that vector: n 32-bit words, entry i = bit pattern of the
 *                    non-negative binary32 maximum of tensor i (bit patterns of non-negative floats order like
 *                    unsigned integers).  Between begin and end the caller takes the element-wise MAXIMUM over
 *                    the ranks that hold shards of the same tensors (one all-reduce with MAX on this vector, on
 *                    the same stream), in place.  Every rank must list the same tensors in the same order.
 *   eco_step_end     pass 2: derive each scale from the (reduced) maximum, quantize, inject, store.
 * With row_offset set in the shards' eco_tensor entries the result is bit-identical to stepping the whole
 * tensors in one context.  Only for ECO_SCALE_PER_TENSOR (other granularities shard with no exchange: use
 * eco_step).  Errors: ECO_ERR_UNSUPPORTED for another granularity; ECO_ERR_INVALID_ARG for eco_step_end
 * without a pending eco_step_begin, or eco_step / eco_step_begin while one is pending; otherwise as eco_step_ex.
 */
eco_status eco_step_begin(eco_ctx* ctx, const eco_hyper* hyper, void* cuda_stream);
eco_status eco_amax_buffer(eco_ctx* ctx, void** device_ptr, size_t* n);
eco_status eco_step_end(eco_ctx* ctx, void* cuda_stream);

/*
 * eco_host_create / eco_host_step / eco_host_destroy -- the step of eco_step (Algorithm 1) for callers
 * that keep the state in HOST memory (offloaded optimizer state).  `tensors` has the layout of
 * eco_tensor but every pointer is a host pointer that must stay valid until eco_host_destroy (pinned
 * memory makes the copies asynchronous and several times faster).
 *   eco_host_create  cuts the list into chunks of whole tensors (about 256 MB of state), allocates three
 *                    device staging slots of the largest chunk's size, three streams, and one eco_ctx per
 *                    chunk.  Errors: as eco_create (the pointers are not required to be device memory).
 *   eco_host_step    for every chunk: copies codes, scales, gradient and moments to its slot, runs the
 *                    kernels of eco_step, copies codes, scales and moments back.  While one chunk is
 *                    stepped the next is copied in and the previous one copied out, so both directions
 *                    of the host link are busy at once.  Returns after everything has been copied back
 *                    and the device-side status of every chunk has been checked.  h2d_bytes / d2h_bytes
 *                    (host, optional) receive the bytes copied in each direction.  The gradient buffers
 *                    are read at every call.  Errors: as eco_step, plus ECO_ERR_TIMEOUT.
 *                    Inside a chunk the staging slot is laid out by kind (all codes, all scales, ...), and
 *                    buffers that follow one another directly in ONE host allocation (a flat pinned buffer
 *                    per kind, tensors back to back, sizes that are multiples of 256 bytes) travel in a single
 *                    copy; anything else is copied buffer by buffer.
 *   eco_host_copies  (host, optional outputs) the number of copies one eco_host_step issues in each
 *                    direction; ECO_ERR_INVALID_ARG for a NULL context.
 *   eco_host_destroy frees all of it (synchronizes the device).  NULL is allowed.
 * eco_step_host is the one-shot form: create, one step, destroy.
 */
eco_status eco_host_create(eco_host_ctx** out, const eco_config* cfg, const eco_tensor* tensors, size_t n, int device);
eco_status eco_host_step(eco_host_ctx* ctx, float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                         uint64_t* h2d_bytes, uint64_t* d2h_bytes);
eco_status eco_host_copies(const eco_host_ctx* ctx, uint64_t* h2d_copies, uint64_t* d2h_copies);
eco_status eco_host_destroy(eco_host_ctx* ctx);
eco_status eco_step_host(const eco_config* cfg, const eco_tensor* tensors, size_t n, int device,
                         float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                         uint64_t* h2d_bytes, uint64_t* d2h_bytes);

/*
 * eco_step_static -- the step of eco_step for ECO_SCALE_PER_TENSOR, for callers that must not
 * allocate device memory.  (The paper has no counterpart: this is a packaging of the same
 * Algorithm 1 arithmetic, not another method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a process whose framework has
 * already reserved the whole device for its own caching allocator, a latency-critical loop that
 * cannot afford the device-wide synchronization an allocation implies, or a host that forbids
 * allocation after start-up.  eco_create allocates its tables and reduction slots with cudaMalloc;
 * this call needs no context and allocates nothing, on the device or through any library.  Its
 * tables and reduction slots live in one fixed array (about 135 KB) inside the loaded library image,
 * which every GPU that loads the library holds until the process exits.
 *
 *   cfg, tensors, n   as eco_create (tensors are device buffers the caller owns); granularity must be
 *                     ECO_SCALE_PER_TENSOR.
 *   lr .. seed        as eco_step.          cuda_stream   as eco_step.
 * Limits: n <= ECO_STATIC_MAX_TENSORS and at most 2^27 parameters in the list (32768 work units of
 * 4096 parameters, each tensor rounded up to whole units); beyond either the call returns
 * ECO_ERR_INVALID_ARG, says so in eco_last_error(NULL), and launches nothing.
 * Behaviour to know about:
 *   - The first call on each device looks up the array's device address (with that device current);
 *     that first call should come before any stream capture.
 *   - All calls share the one array, which still holds the previous call's tables: every call
 *     rewrites what it uses and zeroes its reduction slots first.  Two calls whose GPU work overlaps
 *     (different streams, or different host threads) race on it; serialize them.
 *   - The call returns after cuda_stream has finished this step (it waits for the stream), unlike
 *     eco_step.  Buffers are checked for NULL and alignment only, not for overlap or residency.
 * Results are bit-identical to eco_create + eco_step on the same inputs.
 * Errors: ECO_ERR_UNSUPPORTED (other granularity, unknown enum), ECO_ERR_INVALID_ARG,
 * ECO_ERR_ALIGNMENT, ECO_ERR_CUDA.
 */
#define ECO_STATIC_MAX_TENSORS 64
eco_status eco_step_static(const eco_config* cfg, const eco_tensor* tensors, size_t n, int device,
                           float lr, float beta1, float beta2, float eps, uint64_t step, uint64_t seed,
                           void* cuda_stream);

/*
 * eco_check -- synchronize cuda_stream and report whether any kernel of this context gave up on a
 * device-side wait.  The streaming kernels wait on shared-memory barriers for their asynchronous
 * copies; every such wait is bounded (about two seconds of clock cycles), after which the kernel
 * records a code in the context and exits instead of hanging.
 * Returns ECO_OK, ECO_ERR_TIMEOUT (state of the tensors is then undefined), or ECO_ERR_CUDA.
 */
eco_status eco_check(eco_ctx* ctx, void* cuda_stream);

/*
 * eco_attach_error_buffers -- give every tensor of the context an FP32 buffer [rows*cols] (device,
 * 16-byte aligned, zero before the first step) that each later step fills with the quantization error
 * e_{t+1} = theta~_{t+1} - theta^_{t+1} of every element (Algorithm 2/3, line 2).  Two uses: ECO_INJECT_EXACT
 * reads it back as e_t (Appendix A; without buffers such a context refuses to step), and with any injection
 * it makes the error observable, e.g. for the consecutive-error statistics of Sec. 4.2 (Fig. 2).
 *   e   host array of n device pointers, n = the context's tensor count, in the order of eco_create.
 * Adds 4 bytes written (and, for ECO_INJECT_EXACT, 4 read) per parameter and step.  Synchronizes the device.
 * Errors: ECO_ERR_INVALID_ARG, ECO_ERR_ALIGNMENT, ECO_ERR_CUDA.
 */
eco_status eco_attach_error_buffers(eco_ctx* ctx, float* const* e, size_t n);

/*
 * eco_selftest_wait -- exercise the bounded device-side wait without any fault: launches one warp that
 * waits on a shared-memory barrier nothing will ever arrive on, with a limit of limit_cycles SM clock
 * cycles (1..2e9) instead of the kernels' two seconds.  The wait must expire, record its code and let the
 * kernel end normally; the call then returns what eco_check reports, i.e. ECO_ERR_TIMEOUT when the
 * mechanism works (ECO_OK would mean the wait was not bounded-and-reported), and clears the status word
 * again so that the context stays usable.  Synchronizes cuda_stream.  Must not overlap an eco_step of the
 * same context.  Errors: ECO_ERR_INVALID_ARG, ECO_ERR_CUDA.
 */
eco_status eco_selftest_wait(eco_ctx* ctx, int64_t limit_cycles, void* cuda_stream);

/*
 * eco_selftest_grid_wait -- the same for the one wait between CTAs that the library has: the grid barrier of the
 * single-launch per-tensor step ("fused_tensor").  Two CTAs meet at a barrier that expects a third arrival, with
 * a limit of limit_cycles (1..2e9); the wait must expire, record its code and let the kernel end normally.
 * Returns ECO_ERR_TIMEOUT when the mechanism works; clears the status word again.  Call it between steps.
 */
eco_status eco_selftest_grid_wait(eco_ctx* ctx, int64_t limit_cycles, void* cuda_stream);

/* eco_destroy -- free the context's tables and scratch (synchronizes the device). NULL is allowed. */
eco_status eco_destroy(eco_ctx* ctx);

/* eco_last_error -- text of the last failure of `ctx`, or of the calling thread's last failed
 * call when ctx is NULL.  The pointer stays valid until the next call on that context / thread. */
const char* eco_last_error(const eco_ctx* ctx);

/*
 * eco_quantize -- theta^_0 = q(theta_0): the symmetric quantizer of Sec. 3.1
 * (scale = max|x| / rho per scale block, zero-point 0) used to initialise the
 * quantized state (Appendix A, initialisation).
 *   x      device, in: f32 [rows*cols], 16-byte aligned.
 *   w, scale  device, out: layouts as in eco_tensor.
 *   cfg->optimizer and cfg->injection are ignored; rounding, seed, step and
 *   tensor_id select the rounding exactly as in eco_step (use step 0 for the
 *   initial state).
 * Asynchronous on cuda_stream except for one temporary device allocation when
 * granularity is ECO_SCALE_PER_TENSOR (freed stream-ordered).
 * Errors: as eco_create.
 */
eco_status eco_quantize(const eco_config* cfg, const float* x, int64_t rows, int64_t cols,
                        void* w, void* scale, uint64_t seed, uint64_t step, uint32_t tensor_id,
                        int device, void* cuda_stream);

/*
 * eco_dequantize -- x^ = value(code) * scale (Sec. 3.1, x^ = s y) for a whole tensor: the weights the
 * forward and backward pass of quantized training read.  No master weights are involved: this only
 * expands the stored codes.
 *   w, scale  device, in: layouts as in eco_tensor (cfg gives format, granularity and scale dtype;
 *             optimizer, rounding and injection are ignored).
 *   out       device, out, 16-byte aligned: f32 [rows*cols], or bf16 [rows*cols] when out_bf16 != 0
 *             (the product is then rounded to bf16, nearest even; INT4 values times a bf16 scale and
 *             most FP8 products need the rounding).
 * Asynchronous on cuda_stream.  Errors: as eco_quantize.
 */
eco_status eco_dequantize(const eco_config* cfg, const void* w, const void* scale, int64_t rows, int64_t cols,
                          void* out, int out_bf16, int device, void* cuda_stream);

/*
 * eco_set_option -- process-wide tuning knobs read by the NEXT eco_create:
 *   "l2_group_bytes"  per-tensor scales only: bytes of inputs one pass-1/pass-2 launch pair
 *                     covers (0, the default: one pair for the whole context, which measured
 *                     fastest; -1 = half the L2 size, so that pass 2 re-reads from L2)
 *   "reverse_pass2"   per-tensor scales only: 1 (default) walks pass 2 in the opposite order
 *                     of pass 1 so that it starts with the most recently read data
 *   "use_stream"      1 (default) uses the persistent kernels fed by bulk asynchronous copies
 *                     wherever a tensor consists of whole, aligned 128-element rows; 0 forces
 *                     the direct-load kernels everywhere
 *   "ctas_per_sm"     persistent grid size in CTAs per SM, 1..3; 0 (default) = as many as the kernel is built to
 *                     keep resident (3 for momentum SGD, 2 for Adam)
 *   "fused_tensor"    per-tensor scales only: run both passes in ONE cooperative launch, wave by wave (a wave = whole
 *                     tensors with about an L2's worth of inputs; the grid meets at a bounded barrier between the
 *                     passes of a wave, and pass 2 finds the wave in shared memory and L2).  0 never, 1 always,
 *                     2 (default) when the whole context is a single wave.  eco_step_begin / eco_step_end always
 *                     use two launches (the exchange sits between them)
 *   "wave_bytes"      input bytes of a wave (default 100 MiB; at least 1 MiB)
 *   "row_cluster"     per-row scales only: 1 (default) steps matrix rows of 4224..16384 columns (whole 128-column
 *                     segments) with thread-block clusters of 2..4 CTAs that share a row; 0 sends them to the
 *                     one-CTA-per-row kernel
 * No option changes any result bit.  Errors: ECO_ERR_INVALID_ARG for an unknown name.
 */
eco_status eco_set_option(const char* name, int64_t value);

/* eco_num_launches -- number of kernels one eco_step of this context enqueues. */
int eco_num_launches(const eco_ctx* ctx);

/* eco_version -- "major.minor.patch" of the library. */
const char* eco_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ECO_H_ */
