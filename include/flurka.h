/*
 * flurka.h -- C ABI of the FLuRKA attention forward pass for NVIDIA B200 (sm_100a).
 *
 * The operation (arxiv 2306.15799, Section 3, Eq. (2), with the row normalisation that
 * Appendix D writes out for kernel attention), per batch b and head h, non-causal:
 *
 *     K' = E K            V' = F V                  (Section 2.1: E, F are k x N, shared)
 *     O  = phi(Q) ( phi(K')^T V' )  /  phi(Q) ( phi(K')^T 1_k )          (row-wise division)
 *
 * with the feature map phi chosen by `variant` (Section 4's instances):
 *     FLURKA_PERFORMER  phi(x)_i = exp(w_i . x - |x|^2 / 2) / sqrt(m),  i < m   (positive random
 *                       features; W = [w_0 .. w_{m-1}] is an input),
 *     FLURKA_RNN        phi(x)_c = elu(x_c) + 1,  c < d                          (no W, m ignored).
 * The per-head linear maps W^Q, W^K, W^V of Eq. (2) are applied by the caller ((E K) W^K = E (K W^K)).
 * No softmax scale is applied: callers pre-scale Q and K.
 *
 * Layout.  All tensors are dense, row-major, contiguous:
 *     Q, K, V, out : [B, H, N, d]      E, F : [k, N]      W : [m, d]
 * (E, F: [H, k, N] with FLURKA_EF_PER_HEAD or-ed into `variant` -- Theorem 1 states the method with
 * one projection pair E_i, F_i per head; they are still shared over the batch)
 * and share one element type per call: bfloat16 (default) or float32 (FLURKA_IO_FP32 or-ed into
 * `variant`).  Accumulation is fp32 in both cases.  With FLURKA_LAYOUT_BNHD or-ed into `variant`,
 * Q, K, V and out are [B, N, H, d] instead: the heads of one position side by side, which is how a
 * model's projections leave them (Eq. (2) treats the heads independently either way).
 *
 * Ownership.  Every pointer is caller-owned; the library keeps none of them after the call returns.
 * `out` must not overlap an input.  Scratch memory comes from the workspace (see below).
 *
 * Errors.  Every function returns FLURKA_OK (0) or a negative flurka_status; on error NOTHING has been
 * launched or copied.  No exceptions, no abort, nothing is printed.
 *
 * Threads and devices.  One call at a time per device (each device has its own workspace, staging
 * buffers and descriptor cache, looked up by the device that is current at the call; the settings
 * made by flurka_set_path, flurka_set_cta_limit and flurka_set_stage_timing are process-wide).
 */
#ifndef FLURKA_H_
#define FLURKA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FLURKA_VERSION 100

typedef enum {
  FLURKA_PERFORMER = 0, /* Linformer-Performer: FAVOR+ positive random features (Section 2.1, Section 4) */
  FLURKA_RNN = 1        /* Linformer-RNN: phi(x) = elu(x) + 1 (Section 2.1, Section 4)                  */
} flurka_kernel_t;

#define FLURKA_IO_BF16 0x000 /* default element type of Q, K, V, E, F, W, out */
#define FLURKA_IO_FP32 0x100 /* or-ed into `variant`: all of them are float32 */
#define FLURKA_LAYOUT_BNHD 0x200 /* or-ed into `variant`: Q, K, V, out are [B,N,H,d], not [B,H,N,d] */
#define FLURKA_EF_PER_HEAD 0x400 /* or-ed into `variant`: E, F are [H,k,N], a pair E_i, F_i per head (Theorem 1) */

typedef enum {
  FLURKA_OK = 0,
  FLURKA_ERR_NULL = -1,        /* a required pointer is NULL                                        */
  FLURKA_ERR_VARIANT = -2,     /* unknown kernel, element type or selector                          */
  FLURKA_ERR_SHAPE = -3,       /* a size is <= 0, d > 128, k > 4096, or the forced path cannot run it */
  FLURKA_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned                                  */
  FLURKA_ERR_WORKSPACE = -5,   /* caller workspace too small, or the library could not allocate one */
  FLURKA_ERR_CUDA = -6,        /* a CUDA call failed; flurka_last_cuda_error() has the cudaError_t  */
  FLURKA_ERR_DEVICE = -7,      /* no sm_100 device is current                                       */
  FLURKA_ERR_OVERLAP = -8,     /* out overlaps an input                                             */
  FLURKA_ERR_TOO_LARGE = -9    /* flurka_forward_static_scratch: scratch need exceeds the built-in array */
} flurka_status;

/* Execution paths, for flurka_set_path().  AUTO picks the tensor-core path when the shape allows. */
typedef enum {
  FLURKA_PATH_AUTO = 0,
  FLURKA_PATH_SIMT = 1,   /* fp32 CUDA-core kernels: any shape within the limits, both element types */
  FLURKA_PATH_TENSOR = 2, /* tcgen05 / TMEM / TMA kernels: bf16 only, shape rules below; else error  */
  FLURKA_PATH_TENSOR_STAGE1 = 3, /* for bisecting: tensor-core down-projection, the rest on CUDA cores */
  FLURKA_PATH_TENSOR_STAGE3 = 4, /* for bisecting: tensor-core query side, the rest on CUDA cores      */
  FLURKA_PATH_TENSOR_STAGE23 = 5 /* for bisecting: tensor-core key and query side, CUDA-core stage 1   */
} flurka_path_t;

/*
 * flurka_forward -- the whole forward pass of Eq. (2) on DEVICE buffers, asynchronous on `stream`.
 *
 *   Q, K, V   device, [B,H,N,d]          E, F   device, [k,N]          W   device, [m,d] (NULL for RNN)
 *   variant   flurka_kernel_t | FLURKA_IO_BF16 / FLURKA_IO_FP32 [| FLURKA_LAYOUT_BNHD] [| FLURKA_EF_PER_HEAD]
 *   out       device, [B,H,N,d], same element type
 *   stream    a cudaStream_t passed as void*; NULL is the default stream
 *
 * Shape limits: B, H, N >= 1, B*H <= 65535; 1 <= d <= 128; 1 <= k <= 4096; PERFORMER: m >= 1.
 * Pointers 16-byte aligned.  The tensor-core path additionally needs bf16, d in {64, 128},
 * N % 8 == 0, k % 64 == 0 with k <= 512, and (PERFORMER) m in {64, 128, 192, 256}; other shapes run
 * on the SIMT path.  The call enqueues work and returns; it never synchronises.  Scratch comes from the
 * workspace set by flurka_set_workspace(), or from one the library obtains on first need and re-uses:
 * when a later problem needs more, the old block is released and a larger one obtained in stream order
 * on `stream` (cudaFreeAsync / cudaMallocAsync), so calls that share the library-owned workspace must
 * be ordered one after the other by the caller, and a call that grows it should not sit inside a
 * stream capture (hand over a workspace with flurka_set_workspace() for that).
 */
int flurka_forward(const void* Q, const void* K, const void* V, const void* E, const void* F,
                   const void* W, int variant, int B, int H, int N, int d, int k, int m, void* out,
                   void* stream);

/*
 * flurka_forward_host -- the same operation (Eq. (2)) on HOST buffers (same shapes and element types).
 * Copies the inputs to the device (cudaMemcpyAsync; pinned host memory makes them asynchronous),
 * runs flurka_forward, copies `out` back and synchronises `stream` before returning.  Larger calls go
 * through the heads in up to eight groups, so that the output of one group is copied back (on a second,
 * library-owned stream) while the inputs of the next are copied in; flurka_last_status() then covers all
 * groups, flurka_debug_copy() the last one.  Device staging buffers are allocated by the library on
 * first use and re-used while they are large enough.
 */
int flurka_forward_host(const void* Q, const void* K, const void* V, const void* E, const void* F,
                        const void* W, int variant, int B, int H, int N, int d, int k, int m, void* out,
                        void* stream);

/*
 * flurka_forward_fused -- Eq. (2) with its per-head linear maps inside the call:
 *
 *     Head_h = phi(Xq W^Q_h) ( phi((E Xk) W^K_h)^T ((F Xv) W^V_h) ),  rows normalised as in Appendix D,
 *     out    = Concat(Head_1 .. Head_H)                                           (Section 2)
 *
 * in the order Section 3 argues for and Appendix B's step list counts ("Linear Transformations":
 * N d_m^2 + 2 d_k d_m^2 instead of 3 N d_m^2): the un-projected keys and values are contracted along
 * the sequence first, W^K and W^V touch only the k contracted rows, W^Q maps the N queries.
 *
 *   Xq, Xk, Xv  device, [B,N,dm]   the layer's inputs before the maps (they may be one and the same buffer)
 *   E, F        device, [k,N]      W  device, [m,d] (NULL for RNN)
 *   Wq, Wk, Wv  device, [dm, H*d]  columns h*d .. h*d+d-1 are head h's map (x W, row vector times matrix)
 *   variant     flurka_kernel_t | FLURKA_IO_BF16 / FLURKA_IO_FP32   (FLURKA_LAYOUT_BNHD is refused: the
 *               layout is fixed)
 *   out         device, [B,N,H,d] = [B,N,H*d], same element type; must not overlap an input
 *
 * Limits as for flurka_forward, and 1 <= dm <= 16384.  The tensor-core path needs what flurka_forward's
 * needs and dm % 64 == 0; everything else runs on CUDA cores.  Asynchronous on `stream`; scratch (the
 * inner problem's, the contracted rows and Xq W^Q as [B,N,H,d]) comes from the workspace as described
 * for flurka_forward, flurka_fused_workspace_bytes() says how much.  Afterwards flurka_last_status,
 * flurka_last_path, flurka_last_launches, flurka_debug_copy (K' and V' after the maps) and, with timing
 * on, flurka_last_stage_ms (stage 0 = contraction and all three linear maps) describe this call.
 */
int flurka_forward_fused(const void* Xq, const void* Xk, const void* Xv, const void* E, const void* F,
                         const void* Wq, const void* Wk, const void* Wv, const void* W, int variant, int B, int H,
                         int N, int dm, int d, int k, int m, void* out, void* stream);
size_t flurka_fused_workspace_bytes(int variant, int B, int H, int N, int dm, int d, int k, int m);

/*
 * A forward pass sharded over the SEQUENCE (several GPUs, each holding a slice of the positions; the
 * paper's own runs spread a model over four GPUs, Section 4).  K' = E K and V' = F V (Eq. (2)) are sums
 * over positions, so a shard computes its part from its slice of K, V and the matching COLUMNS of E, F,
 * the parts are added over the shards, and everything after is local to a shard's queries:
 *
 *   flurka_forward_partial   K, V: device [B,H,n,d] (or [B,n,H,d]), the shard's n positions; E, F: device
 *                            [k,n], the matching columns as a dense matrix.  Leaves this shard's part of
 *                            K', V' in the workspace (fp32, [2][B*H][k][d]).
 *   flurka_partial_sums      Where that block is (device pointer, bytes).  The CALLER adds it over the
 *                            shards in place -- an all-reduce (sum) of that many bytes, e.g. NCCL on the
 *                            same stream -- which is the only exchange between the GPUs.
 *   flurka_forward_finish    Q: device, the shard's queries (n may differ from the first call's), W, out:
 *                            the key side and the query side on the summed K', V'.
 *
 * Variant word, shape limits, alignment, streams and errors as for flurka_forward; the three calls use
 * the current device's workspace, so nothing else may run on it in between.  flurka_forward_finish
 * returns FLURKA_ERR_WORKSPACE when no matching flurka_forward_partial came before it.
 */
int flurka_forward_partial(const void* K, const void* V, const void* E, const void* F, int variant, int B, int H,
                           int N, int d, int k, int m, void* stream);
int flurka_partial_sums(void** dev_ptr, size_t* bytes);
int flurka_forward_finish(const void* Q, const void* W, int variant, int B, int H, int N, int d, int k, int m,
                          void* out, void* stream);

/*
 * flurka_backward -- the gradients of flurka_forward's output (the method is one for training, Sections 1
 * and 4; the paper prints no backward formulas, these follow from Eq. (2) and Appendix D by the chain rule):
 * given dO = d loss / d out, writes d loss / d Q, K, V (shapes of Q, K, V) and d loss / d E, F (shape of E,
 * F: summed over every batch and head that shares the pair).  W is not learned and gets no gradient.
 * All buffers are DEVICE buffers of the call's element type; variant word, layouts, limits, alignment,
 * stream and workspace rules as for flurka_forward (flurka_backward_workspace_bytes says how much scratch).
 * The forward's key-side summaries are recomputed inside the call, so nothing has to be kept from the
 * forward pass.  No output may overlap an input or another output.
 * Kernels: where flurka_forward's tensor-core path takes the shape (bf16, the rules below) the two
 * down-projections, the key-side summaries and, with E, F shared by the heads, the gradients dK, dV, dE, dF
 * (products with E, F, K, V: dK', dV' enter as two bf16 terms) run on tcgen05 kernels; so does the query side
 * (dQ and the gradients of the key-side summaries) for d = 64 and, PERFORMER only, d = 128, and the key side's
 * backward half (dK', dV' from those gradients) for PERFORMER with d = 64.
 * flurka_last_path() then reports FLURKA_PATH_TENSOR (query side included) or FLURKA_PATH_TENSOR_STAGE1.
 * Everything else, and every shape under FLURKA_PATH_SIMT, runs on CUDA cores with fp32 arithmetic;
 * FLURKA_PATH_TENSOR forced on a shape without a tensor-core query side returns FLURKA_ERR_SHAPE.
 */
int flurka_backward(const void* Q, const void* K, const void* V, const void* E, const void* F, const void* W,
                    const void* dO, int variant, int B, int H, int N, int d, int k, int m, void* dQ, void* dK,
                    void* dV, void* dE, void* dF, void* stream);
size_t flurka_backward_workspace_bytes(int variant, int B, int H, int N, int d, int k, int m);

/* Bytes of device scratch flurka_forward needs for this problem (0 on invalid arguments). Holds the
 * fp32 projections K', V' (Eq. (2)'s E K and F V), the key-side feature summaries and a status word. */
size_t flurka_workspace_bytes(int variant, int B, int H, int N, int d, int k, int m);

/* Hands the library a caller-owned device workspace (256-byte aligned) for the current device.
 * NULL/0 returns to the library-owned one. The caller keeps it alive until the last call using it
 * has finished. */
int flurka_set_workspace(void* dev_ptr, size_t bytes);

/* Forces an execution path for later calls (flurka_path_t); returns the previous one. */
int flurka_set_path(int path);

/* Tuning / test knob: the persistent tensor-core kernels use at most `max_ctas` CTAs (0 = one per SM,
 * the default), so that small problems still exercise several tiles per CTA. Returns the old limit. */
int flurka_set_cta_limit(int max_ctas);

/* Tuning / test knob: whether the tensor-core down-projection (Eq. (2)'s E K, F V) may run as pairs of
 * CTAs that share the K / V tiles (the default, used when k % 256 == 0, B*H*d % 256 == 0 and E, F are
 * shared by the heads) or always as single CTAs.  Returns the old setting. */
int flurka_set_stage1_pairs(int on);

/* The path the most recent successful flurka_forward (or flurka_backward) took (never FLURKA_PATH_AUTO). */
int flurka_last_path(void);

/* Number of kernels the most recent successful flurka_forward launched. */
int flurka_last_launches(void);

/*
 * Copies an intermediate of the most recent flurka_forward to a DEVICE buffer, asynchronously on
 * `stream` (order it after the forward).  `which`: 0 = K' [B,H,k,d] fp32, 1 = V' [B,H,k,d] fp32
 * (Eq. (2)'s E K, F V), 2 = key-side summary a [B,H,p,d] fp32 (a_i = sum_j phi(k'_j)_i v'_j / z_i,
 * p = m or d; only on paths whose query side runs on CUDA cores), 3 = per-feature weights [B,H,p] fp32 (PERFORMER: log z_i with the
 * exponent maximum added back; RNN: z_i), 4 = status words (4 x int32).  `bytes` must equal the
 * intermediate's size.
 */
int flurka_debug_copy(int which, void* dev_dst, size_t bytes, void* stream);

/* Synchronises the device and returns the status word the kernels of the last call left behind:
 * 0 = clean; bit 0 = a bounded wait gave up (results invalid). */
int flurka_last_status(void);

/* cudaError_t (as int) behind the most recent FLURKA_ERR_CUDA. */
int flurka_last_cuda_error(void);

/*
 * Per-stage device timing.  With timing on, flurka_forward records CUDA events on its stream before
 * and after each of the three stages of Eq. (2): 0 = down-projection (E K, F V), 1 = key side
 * (phi(K'), phi(K')^T V', phi(K')^T 1), 2 = query side (phi(Q), the product, the division).
 * flurka_last_stage_ms waits for the last forward and writes the three durations in milliseconds;
 * it returns FLURKA_ERR_WORKSPACE if that forward ran with timing off.
 */
int flurka_set_stage_timing(int on);
int flurka_last_stage_ms(float* ms3);

/*
 * Measurement aid for the roofline of the query side, whose N * m exponentials per head (the feature
 * map phi(Q) of Section 2.1) go through the special-function unit, a limit that FLOP and byte counts
 * do not show.  Runs a kernel of nothing but independent ex2.approx chains on every SM of the current
 * device (default stream, a few milliseconds, synchronises) and writes the rate it reached, in 1e9
 * exponentials per second, to the HOST double `gexp_per_s`.
 */
int flurka_measure_ex2_rate(double* gexp_per_s);

/* Static, human-readable text for a flurka_status. */
const char* flurka_strerror(int code);

/* FLURKA_VERSION of the loaded library. */
int flurka_version(void);

/*
 * flurka_forward_static_scratch -- flurka_forward for callers that are not allowed to allocate.
 * (A convenience of this library; the paper has no counterpart.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework whose caching
 * allocator owns all device memory and forbids side allocations, in a latency-critical serving loop
 * where an allocation would stall the device, or in a sandboxed plug-in that is only handed finished
 * buffers.  flurka_forward may call cudaMalloc for its workspace on first use (unless the caller set
 * one); this entry point never calls cudaMalloc, cudaFree or any allocating routine.  Its scratch
 * (the fp32 projections K', V', the key-side summaries and a status word) sits in a device array of
 * FLURKA_STATIC_SCRATCH_BYTES that is compiled into the library, so every GPU that loads the
 * library carries those bytes until the process exits.
 *
 * Arguments, layouts, element types and error codes are those of flurka_forward; inputs and `out`
 * are still the caller's device buffers.  Differences:
 *   - a problem whose flurka_static_scratch_need() exceeds FLURKA_STATIC_SCRATCH_BYTES is refused
 *     with FLURKA_ERR_TOO_LARGE and nothing is launched (that need is a little below
 *     flurka_workspace_bytes(), which also reserves room only the tensor-core kernels use);
 *   - it always runs the fp32 CUDA-core kernels (flurka_set_path is ignored), and it does not feed
 *     flurka_debug_copy / flurka_last_status / flurka_last_path / flurka_last_stage_ms, which keep
 *     describing the last flurka_forward;
 *   - the first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current); make that first call outside any stream capture;
 *   - all calls share the one array and it keeps what the last call left there.  The call itself
 *     clears what has to start at zero, but two calls that overlap in time on the GPU (different
 *     streams, or this one next to another thread's) race on it: serialise them.
 */
#define FLURKA_STATIC_SCRATCH_BYTES (8u << 20)
/* Bytes of the built-in array flurka_forward_static_scratch would use for this problem (0 on invalid
 * arguments).  (Like the entry point itself, without a counterpart in the paper.) */
size_t flurka_static_scratch_need(int variant, int B, int H, int N, int d, int k, int m);
int flurka_forward_static_scratch(const void* Q, const void* K, const void* V, const void* E,
                                  const void* F, const void* W, int variant, int B, int H, int N,
                                  int d, int k, int m, void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FLURKA_H_ */
