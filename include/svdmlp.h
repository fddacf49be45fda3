/*
 * svdmlp.h - C ABI of libsvdmlp: forward pass of a SwiGLU MLP whose gate, up and down weights
 * are stored as rank-r SVD factors, for NVIDIA B200 (sm_100a).
 *
 * Notation (nn.Linear style): a weight W[out, in] ~= U[out, r] * V[r, in]; a projection is the
 * low-rank chain  y = (x V^T) U^T.  In the paper's kernel notation (Section 4.2.1, O = X U V
 * with U[K x r], V[r x N]) the paper's U is this V^T and the paper's V is this U^T; M = T.
 *
 * Unless a parameter says HOST, every pointer is a DEVICE pointer to a contiguous row-major
 * array; factor tensors and X are bf16.  Base pointers must be 16-byte aligned and d, ffn and
 * the ranks multiples of 8.  The caller owns every buffer it passes; a handle borrows the six
 * factor pointers (they must stay valid and unchanged until svdmlp_destroy) and owns its
 * workspace.  Every entry point returns an svdmlp_status (0 = ok, negative = error); nothing
 * throws, aborts or traps.  Shape and pointer errors are detected on the host before any
 * launch.  Forward calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 * the default stream) and never synchronise the host unless stated.  There is no CPU fallback:
 * on a machine without an sm_100 device create/forward return SVDMLP_ERR_ARCH / SVDMLP_ERR_CUDA.
 * One handle must not be used from two streams at once (its workspace is shared).
 */
#ifndef SVDMLP_H_
#define SVDMLP_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct svdmlp svdmlp_t; /* opaque */

typedef enum {
    SVDMLP_OK = 0,
    SVDMLP_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, T > max_T ...              */
    SVDMLP_ERR_UNSUPPORTED = -2, /* a shape the selected path cannot run                         */
    SVDMLP_ERR_ALIGNMENT = -3,   /* pointer not 16-byte aligned or a dimension not multiple of 8 */
    SVDMLP_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed                            */
    SVDMLP_ERR_ARCH = -5,        /* current device is not compute capability 10.x                */
    SVDMLP_ERR_NOMEM = -6,       /* workspace allocation failed / caller workspace too small     */
    SVDMLP_ERR_TIMEOUT = -7      /* a bounded device-side wait gave up (see last_device_status)  */
} svdmlp_status;

/* svdmlp_create flags */
#define SVDMLP_FLAG_Y_FP32 0x1u      /* Y is written as fp32 instead of bf16                      */
#define SVDMLP_FLAG_PATH_SKINNY 0x10u /* force the weight-streaming (small-T) kernels for every T */
#define SVDMLP_FLAG_PATH_TENSOR 0x20u /* force the tcgen05 (large-T) kernels for every T          */
#define SVDMLP_FLAG_NO_CTA_PAIRS 0x80u /* large T: single-CTA tcgen05 kernels only (no cta_group::2 pairs)      */
#define SVDMLP_FLAG_DECODE_REGISTERS 0x40u /* small T: three register-streaming kernels, not the persistent one */
#define SVDMLP_FLAG_NO_TMEM_STRIP 0x100u /* large T, ranks <= 256: gate/up with the Z strip in shared memory, not TMEM */
#define SVDMLP_FLAG_DECODE_COOPERATIVE 0x400u /* small T: cooperative launch of the persistent kernel (residency guaranteed by the driver) instead of a programmatic dependent launch */
#define SVDMLP_FLAG_TOKEN_SLABS 0x800u /* large T: gate/up and the first down product run over token slabs whose H (64 MB) stays in L2; off by default (slower as measured) */
#define SVDMLP_FLAG_NO_FUSED_DOWN1 0x1000u /* large T, ranks <= 128: gate/up and the first down product as two kernels with H in global memory, not the one fused kernel */
#define SVDMLP_FLAG_NO_CLUSTER_SPLITK 0x2000u /* large T: split-K sums through fp32 partials and a reduction launch, never through distributed shared memory inside a cluster */
#define SVDMLP_FLAG_NO_WIDE_GATEUP 0x200u /* large T, ranks > 256: gate/up on 128-wide tiles, not 256-wide ones */

/*
 * Create a handle for one factored MLP layer (Algorithm 2's operands: gate/up factors of rank
 * r_gate/r_up and down factors of a separate rank r_down).
 *   Ug[ffn, r_gate] Vg[r_gate, d]   gate:  G  = (X Vg^T) Ug^T
 *   Uu[ffn, r_up]   Vu[r_up, d]     up:    Up = (X Vu^T) Uu^T
 *   Ud[d, r_down]   Vd[r_down, ffn] down:  Y  = ((SiLU(G) .* Up) Vd^T) Ud^T
 * max_T bounds T of later forward calls and sizes the workspace (H slab, narrow intermediates,
 * status word).  The factors are only read.  Work enqueued at create time (workspace clears)
 * goes to `stream`; the call returns after that work has completed.
 * Errors: INVALID_ARG, ALIGNMENT, ARCH, NOMEM, CUDA.  On error *out is NULL.
 */
int svdmlp_create(svdmlp_t** out, int d, int ffn, int r_gate, int r_up, int r_down,
                  const void* Ug, const void* Vg, const void* Uu, const void* Vu,
                  const void* Ud, const void* Vd, int max_T, unsigned flags, void* stream);

/*
 * Y[T, d] = MLP(X[T, d])  (Algorithm 2; Algorithm 3 is its gate+up stage):
 *   Zg = X Vg^T, Zu = X Vu^T            (narrow, kept on chip / in the handle's workspace)
 *   H  = SiLU(Zg Ug^T) .* (Zu Uu^T)     SiLU(g) = g / (1 + e^-g)
 *   Y  = (H Vd^T) Ud^T
 * X bf16; Y bf16 (fp32 with SVDMLP_FLAG_Y_FP32).  Products accumulate in fp32.  1 <= T <= max_T.
 * The kernels are chosen from T and the ranks: weight-streaming kernels up to 8 tokens, and up to 32
 * tokens where the one-kernel decode path fits the shape (ranks 1024: up to 16); tcgen05 kernels
 * otherwise.  Reproducibility: the tcgen05 kernels sum in a fixed order, so repeated calls on the same inputs give
 * the same bits; the weight-streaming kernels reduce Zd over the ffn slices with fp32 atomic adds, whose order is
 * not fixed, so their outputs can differ between calls in the last bits (fp32 rounding of a 148-term sum, far
 * inside the bf16 rounding of Y for most elements).  Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, CUDA.
 */
int svdmlp_forward(svdmlp_t* h, const void* X, int T, void* Y, void* stream);

/*
 * Same computation with HOST buffers: X_host[T, d] bf16 is copied to the device, the forward
 * runs, Y is copied back to Y_host, all on `stream`, and the call waits for the stream before
 * returning.  For full copy overlap the host buffers should be page-locked.  On a non-default stream the
 * three operations of a call are recorded as one graph, which later calls with the same X_host, Y_host
 * and T replay (one launch instead of three); the buffers' contents may of course change between calls.
 * The first call allocates the device-side staging copies of X and Y ([max_T, d] each).
 */
int svdmlp_forward_host(svdmlp_t* h, const void* X_host, int T, void* Y_host, void* stream);

/*
 * One pre-norm residual layer of a stack of factored MLPs (the 40-layer configuration):
 *   h_out = h_in + MLP(RMSNorm(h_in)),  RMSNorm(h)[t, :] = h[t, :] / sqrt(mean(h[t, :]^2) + eps)
 * with unit norm weight.  h_in, h_out are fp32 [T, d] (the residual stream stays fp32; the
 * normalised rows are rounded to bf16 as the MLP input).  h_out may alias h_in.
 * For T <= 8 normalisation and residual add run inside the decode kernel.  Otherwise the normalised
 * rows pass through a [max_T, d] bf16 buffer that the first such call allocates (cudaMalloc may
 * synchronise the device, so make that call before any stream capture).
 */
int svdmlp_forward_prenorm_residual(svdmlp_t* h, const float* h_in, float* h_out, int T,
                                    float eps, void* stream);

/*
 * The two halves of the forward pass for tensor parallelism over ffn (Section 4.2.2, last paragraph, and
 * Figure 4: gate and up projections partitioned by columns, the down projection by rows, one all-reduce).  With
 * factored weights the partition falls on the rank-r chain: shard g of G holds the rows Ug[F_g, :], Uu[F_g, :]
 * and the columns Vd[:, F_g] of its slice F_g of ffn (as contiguous arrays; a handle is created on them with
 * ffn = |F_g|), and Vg, Vu, Ud whole.  Then  Zd = sum_g Zd_g  with  Zd_g = H[:, F_g] Vd[:, F_g]^T,  so what the
 * ranks exchange is the narrow fp32 Zd[T, r_down] (r_down / d of the bytes of the paper's all-reduce of Y), and
 * every rank finishes with the replicated Ud:
 *   svdmlp_forward_partial  Zd_out[T, r_down] (fp32) = (SiLU((X Vg^T) Ug^T) .* ((X Vu^T) Uu^T)) Vd^T   of this handle
 *   (the caller sums Zd_out over the shards: an all-reduce)
 *   svdmlp_forward_finish   Y[T, d] = Zd Ud^T,  Zd fp32 [T, r_down] (rounded to fp16 as the product's operand for T > 32)
 * Both are asynchronous on `stream`.  svdmlp_forward_partial followed by svdmlp_forward_finish on the same handle
 * with nothing added in between equals svdmlp_forward.  Where svdmlp_forward streams the weights (T <= 32) the pair runs on the register-streaming
 * decode kernels (the one-kernel decode path cannot stop half way).  Errors as svdmlp_forward.
 */
int svdmlp_forward_partial(svdmlp_t* h, const void* X, int T, float* Zd_out, void* stream);
int svdmlp_forward_finish(svdmlp_t* h, const float* Zd, int T, void* Y, void* stream);

/*
 * The same pair with the exchange done by the library's own kernels instead of a collective library (Figure 4's
 * AllReduce, on the narrow Zd): every rank pushes its partial into its slot of every peer's receive buffer with
 * plain peer stores and raises one flag per peer; the finishing call waits (bounded) for the flags of the step and
 * sums the slots.  Set-up, by the caller, once: on every rank a receive buffer of svdmlp_tp_recv_bytes(G, max_T,
 * r_down) bytes and G 64-bit flag words, ZEROED, both mapped into every peer (peer access, IPC or symmetric
 * memory); `peers` lists them by rank as this rank addresses them.  Steps are numbered 1, 2, 3, ... and every rank
 * calls push(step) then gather(step), on one stream, for each step in turn (the two-deep buffering relies on it).
 *   svdmlp_forward_partial_push    Zd_g of this shard -> slot `rank` of every rank's buffer; flags[rank] = step
 *   svdmlp_forward_finish_gather   waits for flags[0..G) >= step, Zd = sum of the slots, Y = Zd Ud^T.
 *     recv, flags: THIS rank's buffer and flag words.  A wait that outlasts the limit (2 s unless changed through
 *     svdmlp_tp_wait_limit_ns of svdmlp_bench.h) sets the status word (svdmlp_last_device_status: -7), leaves Y
 *     unspecified and returns normally: nothing spins without bound.
 * G <= 8.  Errors: as svdmlp_forward_partial / svdmlp_forward_finish; INVALID_ARG also for step 0 or a bad rank.
 */
typedef struct svdmlp_tp_peers {
    int world, rank;                 /* G and this rank's index */
    float* recv[8];                  /* recv[p]: rank p's receive buffer, as addressed from this rank */
    unsigned long long* flags[8];    /* flags[p]: rank p's G flag words */
} svdmlp_tp_peers_t;
size_t svdmlp_tp_recv_bytes(int world, int max_T, int r_down);
int svdmlp_forward_partial_push(svdmlp_t* h, const void* X, int T, const svdmlp_tp_peers_t* peers,
                                unsigned long long step, void* stream);
int svdmlp_forward_finish_gather(svdmlp_t* h, float* recv, const unsigned long long* flags, int world,
                                 unsigned long long step, int T, void* Y, void* stream);

/*
 * The paper's XUV operator (Section 4.2.1):  Y[T, out] = (X[T, in] V^T) U^T  with U[out, r],
 * V[r, in]; X, U, V, Y bf16.  `workspace` is caller-owned device scratch of at least
 * svdlinear_workspace_bytes(T, in, out, r) bytes, 256-byte aligned; its contents are
 * overwritten.  Errors: INVALID_ARG, ALIGNMENT, NOMEM (workspace too small), ARCH, CUDA.
 */
int svdlinear_forward(const void* X, int T, int in, int out, int r, const void* U, const void* V,
                      void* Y, void* workspace, size_t workspace_bytes, void* stream);
size_t svdlinear_workspace_bytes(int T, int in, int out, int r);

/*
 * The same operator with a handle (Section 4.2.1; the factors of a layer are fixed at inference time, Section
 * 2.1): svdlinear_create does once what svdlinear_forward repeats on every call for T > 32 - the fp16 re-encoding
 * of U that the second product needs (its first operand, Z, is fp16) and the tensor maps of the factors - and owns
 * the workspace, sized for max_T.  The handle borrows U and V (they must outlive it).  svdlinear_apply computes
 * Y[T, out] = (X V^T) U^T for 1 <= T <= max_T, asynchronously on `stream`.
 * Number range for T > 32 (both entry points): Z = X V^T and the re-encoded U are fp16, so |Z| and |U| must stay
 * below 65504; svdlinear_create checks U and, if a value exceeds the range, svdlinear_apply returns
 * SVDMLP_ERR_UNSUPPORTED for T > 32 (T <= 32 runs on bf16 kernels with fp32 intermediates and has no such limit).
 * svdlinear_forward cannot report the condition (it never synchronises): out-of-range factors give inf/NaN there.
 * Errors: INVALID_ARG, ALIGNMENT, ARCH, NOMEM, CUDA, UNSUPPORTED.
 */
typedef struct svdlinear svdlinear_t; /* opaque */
int svdlinear_create(svdlinear_t** out_handle, int in, int out, int r, const void* U, const void* V, int max_T,
                     void* stream);
int svdlinear_apply(svdlinear_t* h, const void* X, int T, void* Y, void* stream);
/*
 * The same with the layout flags of Algorithm 2's XUV_Kernel (is_XT: the input arrives pre-transposed; req_OT:
 * the output is wanted transposed), so that a caller whose neighbouring operators work on transposed activations
 * needs no transpose pass of its own:
 *   SVDLINEAR_X_TRANSPOSED   X is X^T[in, T] (row-major, T contiguous)
 *   SVDLINEAR_Y_TRANSPOSED   Y is written as Y^T[out, T]
 * With either flag T must be a multiple of 8 (16-byte row pitch).  For T > 32 neither costs a pass over memory:
 * X^T tiles are loaded as they are and multiplied as an MN-major operand, and the epilogue stores transposed
 * tiles.  For T <= 32 the operand (at most 32 rows) passes through a scratch copy.  layout = 0 is svdlinear_apply.
 * Errors: as svdlinear_apply; ALIGNMENT also for T not a multiple of 8 with a flag set.
 */
#define SVDLINEAR_X_TRANSPOSED 0x1u
#define SVDLINEAR_Y_TRANSPOSED 0x2u
int svdlinear_apply_layout(svdlinear_t* h, const void* X, int T, void* Y, unsigned layout, void* stream);
int svdlinear_destroy(svdlinear_t* h);

/*
 * XUV operator without any allocation (the paper has no counterpart: it is a packaging variant
 * of svdlinear_forward for small token counts, not a step of the method).
 *
 * For callers that may not allocate device memory at the point of the call: serving loops whose
 * device memory has been handed in full to a framework's caching allocator (a cudaMalloc there
 * can fail or stall the whole device while it synchronises), and code with a no-allocation rule
 * after start-up.  Such callers also have no spare buffer to lend as `workspace`, so the narrow
 * intermediate Z[T, r] (fp32) lives in a fixed array inside the library instead: every GPU that
 * loads the library holds SVDLINEAR_NOALLOC_MAX_ELEMS * 4 bytes (128 KiB) for it until exit.
 *
 * Same arguments and result as svdlinear_forward minus the workspace.  Limits: T <=
 * SVDLINEAR_NOALLOC_MAX_T, T * r <= SVDLINEAR_NOALLOC_MAX_ELEMS and r <= SVDLINEAR_NOALLOC_MAX_R
 * (the second kernel holds an 8-token strip of Z in shared memory, 32 (r + 32) bytes of the 227 KiB
 * an SM has), otherwise SVDMLP_ERR_UNSUPPORTED is returned and nothing is launched.  The call performs no cudaMalloc,
 * cudaFree or other allocating call.  The first call on each device looks up the device address
 * of the array (one cudaGetSymbolAddress with that device current); make that first call before
 * any stream capture begins.  All calls on a device share the one array: it keeps the previous
 * call's contents, so each call first clears the T * r values it accumulates into (on `stream`),
 * and two calls whose kernels can overlap on the GPU (different streams, no dependency between
 * them) race on it and give wrong results - serialise them.
 */
#define SVDLINEAR_NOALLOC_MAX_T 32
#define SVDLINEAR_NOALLOC_MAX_ELEMS 32768
#define SVDLINEAR_NOALLOC_MAX_R 7232
int svdlinear_forward_noalloc(const void* X, int T, int in, int out, int r, const void* U,
                              const void* V, void* Y, void* stream);

/*
 * Rank selection of the compression front-end (Eq. 5): the rank that stores a [k, n] weight as factors
 * U[k, r], V[r, n] at compression ratio `ratio` (fraction of the dense parameters removed, 0 <= ratio < 1),
 * rounded to a multiple of `block` (the kernels' tile granularity; the paper uses its tensor-engine tile):
 *     r = floor( k n (1 - ratio) / ((k + n) block) + alpha ) * block,     alpha = 0.5 rounds to nearest.
 * Host arithmetic only (no CUDA call).  Returns r (which may be 0 for tiny matrices or ratios near 1), or
 * SVDMLP_ERR_INVALID_ARG for non-positive sizes, a ratio outside [0, 1) or alpha outside [0, 1].
 */
int svdmlp_block_aligned_rank(int k, int n, double ratio, int block, double alpha);

/*
 * Capacity / intensity model of the forward pass on this device: what Section 4.2.1 "Blocking" does with Eq. 10
 * (arithmetic intensity as a function of the row-strip height B_M) and Eq. 11 (peak on-chip usage) for the
 * paper's accelerator, restated for the memories of an sm_100 SM.  Host arithmetic only (no CUDA call, usable
 * without a GPU); it reports the decisions svdmlp_forward takes for the shape, with the numbers behind them.
 *   strip_rows      B_M: token rows that share one pass over the factor tiles (256: the two CTAs of a pair hold
 *                   128 rows each and split every factor chunk; 8/16/32 on the weight-streaming path)
 *   tmem_cols_*     32-bit tensor-memory columns (of 512 per SM) held by the gate/up kernel: the Z strip as packed
 *                   fp16 A operand (r columns for gate + up, ranks <= 256), the fp32 accumulators of G and Up, and -
 *                   fused kernel, ranks <= 128 - the fp32 accumulator of Zd
 *   smem_bytes      shared memory per CTA (of 232448): operand ring, H tile and store staging of that kernel
 *   flops           2 T r (3 d + 3 ffn)   (Section 3's count for the three factored projections)
 *   hbm_bytes       factors once + X in + Y out, plus the write and read of H when it is not fused away and is
 *                   larger than `l2_bytes` (all 16-bit)
 *   sm_bytes        bytes entering the SMs: Eq. 10's denominator generalised to the MLP - X, Y, Z, Zd, H once each
 *                   way, and the factors once per row strip:  s [ 2 T d + ceil(T / B_M) 3 r (d + ffn) + ... ]
 *   intensity_hbm   flops / hbm_bytes;  intensity_sm = flops / sm_bytes (Eq. 10's quantity: it grows with B_M and
 *                   saturates at 2 r / s per projection)
 *   ridge_hbm       tensor_tflops / hbm_gbs in FLOP per byte: above it the shape is bound by the tensor pipe
 *   t_tensor_us, t_hbm_us   flops / tensor_tflops and hbm_bytes / hbm_gbs;  t_floor_us = the larger
 * path: 0 weight-streaming decode kernels, 1 tcgen05 kernels, 2 tcgen05 kernels with gate/up and the first down
 * product fused (H never leaves the SM).  tensor_tflops, hbm_gbs: the peaks to model against (<= 0: 1648 TFLOP/s
 * and 6547 GB/s, measured on a B200); l2_bytes <= 0: 126 MB.  Equal ranks r for the three projections.
 * Errors: INVALID_ARG (non-positive sizes, NULL out).
 */
typedef struct svdmlp_model {
    int d, ffn, r, T;
    int path, strip_rows, z_in_tmem;
    int tmem_cols_strip, tmem_cols_acc, tmem_cols_zd, tmem_cols_total;
    long smem_bytes;
    double flops, hbm_bytes, sm_bytes;
    double intensity_hbm, intensity_sm, ridge_hbm;
    double t_tensor_us, t_hbm_us, t_floor_us;
} svdmlp_model_t;
int svdmlp_model(int d, int ffn, int r, int T, double tensor_tflops, double hbm_gbs, double l2_bytes,
                 svdmlp_model_t* out);

/*
 * Compression front-end on the device (Section 4.1 with S = I, i.e. without the activation-aware whitening, which
 * needs calibration data: Eq. 3 is then the plain SVD W = U Sigma V^T; Eq. 6-8 fold Sigma into the factors).
 * W[out, in] is a dense fp32 weight on the device; the call writes the factors of the r largest singular values,
 *     U_out[out, r] = U_r diag(sigma_r),  V_out[r, in] = V_r^T                    (flags = 0; W ~= U_out V_out), or
 *     U_out = U_r diag(sqrt(sigma_r)),    V_out = diag(sqrt(sigma_r)) V_r^T        (SVDMLP_COMPRESS_SPLIT_SQRT: Eq. 6-7)
 * as bf16 (round to nearest even), ready for svdmlp_create / svdlinear_create.  sigma_out, if not NULL, is a HOST
 * array of min(out, in) floats that receives all singular values in descending order.  r = the value of
 * svdmlp_block_aligned_rank (Eq. 5) or any 1 <= r <= min(out, in).  One-sided Jacobi in fp32 with fp64 dot
 * products: singular values to about 1e-6 relative.  `workspace`: device scratch of at least
 * svdmlp_compress_workspace_bytes(out, in) bytes, 256-byte aligned.  An offline step: the call synchronises
 * `stream` several times (once per sweep) and returns when the factors are written.
 * Errors: INVALID_ARG, ALIGNMENT, NOMEM (workspace too small), ARCH, CUDA.
 */
#define SVDMLP_COMPRESS_SPLIT_SQRT 0x1u
int svdmlp_compress(const float* W, int out, int in, int r, void* U_out, void* V_out, float* sigma_out,
                    void* workspace, size_t workspace_bytes, unsigned flags, void* stream);
size_t svdmlp_compress_workspace_bytes(int out, int in);

/* Free the workspace.  Waits for the device to finish work that uses it.  NULL is allowed. */
int svdmlp_destroy(svdmlp_t* h);

/* Static, human-readable text for a status code. */
const char* svdmlp_strerror(int status);

/*
 * Synchronises the device and returns the status word device code writes when a bounded wait
 * gives up (SVDMLP_OK if none did).  The word is cleared by the call.
 */
int svdmlp_last_device_status(svdmlp_t* h);

#ifdef __cplusplus
}
#endif
#endif /* SVDMLP_H_ */
