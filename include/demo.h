/*
 * demo.h -- C ABI of the B200-native DeMo optimizer transform (arXiv 2411.19870).
 *
 * One optimizer step of the paper's Algorithm 1 ("DeMo: Decoupled Momentum") is
 *     for every simulated worker w:   demo_compress(ctx, w, grads_w, momentum_w, payload_w, stream)
 *     once:                           demo_decode_apply(ctx, payloads, W, params, stream)
 * All tensors live in device memory owned by the caller; the library owns only its context
 * (DCT tables, chunk tables, pointer tables, one status word).  Every call enqueues work on the
 * given CUDA stream and returns; argument errors are reported synchronously before any launch,
 * device-side problems through demo_device_status().  No C++ exception crosses this boundary,
 * there is no global state and no CPU fallback: without a CUDA device every compute entry point
 * fails with DEMO_ERR_CUDA.
 *
 * Streams: when a context holds both 2-D and 1-D tensors, the small kernel of the 1-D tensors runs on a
 * stream of the context beside the kernel of the 2-D tensors: it starts after everything already queued on
 * cuda_stream and cuda_stream continues only when it has finished, so the caller sees plain stream order.
 *
 * CUDA graphs: demo_compress and demo_decode_apply copy their pointer arrays to device tables only
 * when a pointer differs from the previous call with the same worker index.  After one ordinary call
 * with the same buffers they enqueue kernel launches only and may be captured into a CUDA graph on
 * the capturing stream; the graph is valid while the buffers and the context live and the context's
 * settings (learning rate, alpha, decode mode, basis, path) are those of the capture.
 *
 * Notation (the paper's): s chunk size, k coefficients kept per chunk, M = s*s (2-D tensors) or
 * s (1-D tensors) elements per chunk, k_eff = min(k, M), W workers, beta momentum decay,
 * lr learning rate (eta), weight_decay (lambda).
 *
 * Payload layout (part of the bit-exact contract; the paper leaves "encode" open, Section 2.1 and
 * the appendix algorithm): for every tensor in descriptor order, for every chunk in row-major
 * order over the chunk grid (c0, c1) of the blocking operator (appendix B.1.2), k_eff records of
 *     struct { int32_t idx; float val; }      little-endian, 8 bytes
 * with idx the flat position inside the chunk (i*s + j for 2-D tiles, j for 1-D segments),
 * records sorted by ascending idx.  Ties at the k-th magnitude go to the lowest idx.
 */
#ifndef DEMO_H_
#define DEMO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct demo_ctx demo_ctx; /* opaque, library-owned */

typedef enum {
    DEMO_OK = 0,
    DEMO_ERR_INVALID_ARG = 1, /* null pointer, bad worker index, misaligned buffer, bad count     */
    DEMO_ERR_SHAPE = 2,       /* order not supported, or a dimension not a multiple of its chunk   */
    DEMO_ERR_K = 3,           /* k < 1 or k > s*s (demo_init_nd: k > DEMO_ND_MAX_CHUNK_ELEMS)      */
    DEMO_ERR_UNSUPPORTED = 4, /* s not in {8,16,32,64,128}, unknown dtype, too many tensors        */
    DEMO_ERR_ALLOC = 5,       /* host or device allocation failed                                  */
    DEMO_ERR_CUDA = 6,        /* a CUDA runtime call failed (no device, launch error, ...)         */
    DEMO_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired                                */
    DEMO_ERR_PAYLOAD = 8      /* decode met a record whose idx is outside its chunk (skipped)      */
} demo_status;

typedef enum { DEMO_F32 = 0, DEMO_BF16 = 1 } demo_dtype;

/* A contiguous row-major tensor: ndim 1 (shape[0] elements) or ndim 2 (shape[0] x shape[1]). */
typedef struct {
    int32_t ndim;
    int64_t shape[2];
} demo_tensor_desc;

/* Hyper-parameters of Algorithm 1's "Require" line. */
typedef struct {
    float beta;            /* momentum decay, m <- beta*m + g                        */
    int32_t chunk;         /* s: 2-D tensors use s x s tiles, 1-D tensors length-s    */
    int32_t topk;          /* k per chunk, 1 <= k <= s*s                              */
    float lr;              /* eta                                                     */
    float weight_decay;    /* lambda, applied to every tensor                         */
    int32_t num_workers;   /* W, number of payloads demo_decode_apply aggregates      */
    int32_t grad_dtype;    /* demo_dtype of the gradient tensors (momentum/params: f32) */
} demo_config;

/* Kernel family used for 2-D tensors.  AUTO picks the register-resident fast-DCT kernels where
 * they exist (s in {32, 64}) and the generic dense-contraction kernels elsewhere; GENERIC forces
 * the latter everywhere (used by tests to cross-check the two).  Both are CUDA paths. */
typedef enum { DEMO_PATH_AUTO = 0, DEMO_PATH_GENERIC = 1 } demo_path;

/*
 * demo_init -- validate the configuration and the tensor list, build the orthonormal DCT-II basis
 * of dimension s (Section 2.1: "precomputed only once before training"), the chunk tables of the
 * blocking operator (appendix B.1.2) and the payload offsets, and allocate the context's small
 * device tables on `cuda_device`.
 *   out        host pointer receiving the context (set to NULL on failure)
 *   cfg        host pointer, read during the call
 *   tensors    host array of n_tensors descriptors, read during the call
 * Errors: INVALID_ARG (nulls, n_tensors < 1, W < 1, beta/lr/weight_decay not finite), SHAPE, K,
 * UNSUPPORTED, ALLOC, CUDA.
 */
demo_status demo_init(demo_ctx **out, const demo_config *cfg, const demo_tensor_desc *tensors,
                      int32_t n_tensors, int32_t cuda_device);

/*
 * Tensors of any order with rectangular chunks -- the general statement of the method in the paper's
 * appendix ("Multilinear Transforms and Chunk-wise Tensor Blocking"): a tensor of shape
 * n_0 x ... x n_{d-1} with n_a = c_a * s_a is cut by the blocking operator into c_0 * ... * c_{d-1}
 * chunks of shape s_0 x ... x s_{d-1}; the chunk transform is the multilinear product
 * T(B; C_0, ..., C_{d-1}) with the orthonormal DCT-II of dimension s_a on axis a (inverse: the
 * transposes).  The paper's worked example, a 128 x 512 matrix in 16 x 32 blocks, is
 * {ndim 2, shape {128, 512}, chunk {16, 32}}.
 *
 * A descriptor is a contiguous row-major tensor of order ndim (1 .. DEMO_ND_MAX_DIMS) with its own chunk
 * shape: 1 <= chunk[a] <= DEMO_ND_MAX_EXTENT, shape[a] a multiple of chunk[a] (the paper assumes this
 * and gives no rule for remainders), M = product of chunk[] <= DEMO_ND_MAX_CHUNK_ELEMS.
 *
 * demo_init_nd builds a context like demo_init (cfg->chunk is ignored; 1 <= cfg->topk <=
 * DEMO_ND_MAX_CHUNK_ELEMS, k_eff = min(k, M) per tensor).  Every other entry point takes the context
 * unchanged, with these differences: a record's idx is the row-major position inside the chunk
 * (((j_0 * s_1 + j_1) * s_2 + j_2) ...), chunks are ordered row-major over the chunk grid
 * (k_0, ..., k_{d-1}); all tensors run on one family of kernels that apply the transform axis by axis as
 * dense contractions on the CUDA cores (no fast-DCT, tensor-core or side-stream path; demo_set_path has
 * no effect); demo_set_basis, demo_set_basis_gaussian and demo_get_basis return UNSUPPORTED (one basis
 * per chunk extent: only the DCT is built).  A descriptor whose chunk is an s x s tile of its last two axes
 * or a length-s segment of its last axis (all other chunk extents 1) gives the payload layout of demo_init
 * with chunk size s on the tensor flattened to its last two axes / last axis and, up to the fp32 rounding of a
 * different summation order, the same records.
 *
 * When EVERY descriptor is of that form with one common s in {8, 16, 32, 64, 128}, the context is that of
 * demo_init: it is built by demo_init on the flattened tensors (topk above s * s is lowered to s * s, which
 * leaves every k_eff unchanged) and is in every respect such a context -- fast-DCT and tensor-map kernels,
 * demo_set_path, caller-supplied bases, demo_set_momentum_domain.
 * Errors: INVALID_ARG, SHAPE (ndim, chunk[a] < 1, shape[a] not a multiple of chunk[a]), K,
 * UNSUPPORTED (chunk extent or chunk too large, dtype, too many tensors), ALLOC, CUDA.
 */
#define DEMO_ND_MAX_DIMS 4
#define DEMO_ND_MAX_EXTENT 128
#define DEMO_ND_MAX_CHUNK_ELEMS 16384
typedef struct {
    int32_t ndim;
    int64_t shape[DEMO_ND_MAX_DIMS];
    int32_t chunk[DEMO_ND_MAX_DIMS];
} demo_nd_tensor_desc;
demo_status demo_init_nd(demo_ctx **out, const demo_config *cfg, const demo_nd_tensor_desc *tensors,
                         int32_t n_tensors, int32_t cuda_device);

/* Bytes of one worker's payload: sum over tensors of n_chunks * k_eff * 8.  0 if ctx is NULL. */
size_t demo_payload_bytes(const demo_ctx *ctx);

/* Where tensor `tensor` sits inside a payload: index of its first record, its number of chunks
 * and its k_eff.  Any output pointer may be NULL.  Errors: INVALID_ARG. */
demo_status demo_payload_layout(const demo_ctx *ctx, int32_t tensor, int64_t *first_record,
                                int64_t *n_chunks, int32_t *k_eff);

/*
 * demo_compress -- the worker side of Algorithm 1 / CompressChunks for worker `worker`, fused per
 * chunk: m <- beta*m + g; Q = DCT(chunk); keep the k_eff largest |Q| as records;
 * m <- m - IDCT(kept) (momentum subtraction with alpha = 1, Section 2.1 "Momentum Subtraction").
 *   grads        host array of n_tensors DEVICE pointers (dtype cfg.grad_dtype), read-only
 *   momentum     host array of n_tensors DEVICE pointers (fp32), updated in place
 *   payload_out  DEVICE buffer of demo_payload_bytes() bytes, overwritten
 *   cuda_stream  cudaStream_t (NULL = default stream)
 * Device buffers must be 16-byte aligned and must not alias each other.  The pointer arrays are
 * host memory, read during the call and not retained.  Calls on one context must be issued in
 * stream order (one stream, or streams the caller orders).  Gradients or momenta that hold NaN or Inf
 * give unspecified values for the chunks they touch, but every chunk still gets k_eff records with
 * distinct, ascending, in-range indices, other chunks are unaffected and nothing hangs or traps.
 * Errors: INVALID_ARG, CUDA.
 */
demo_status demo_compress(demo_ctx *ctx, int32_t worker, const void *const *grads,
                          float *const *momentum, void *payload_out, void *cuda_stream);

/*
 * demo_decode_apply -- the server side of Algorithm 1 / Decompress&Aggregate plus the update,
 * fused per chunk: S = sum over the n_payloads payloads (in the order given) of their records;
 * R = IDCT(S); x <- x - lr * (sign(R) + weight_decay * x), with sign(0) = 0.
 *   payloads     host array of n_payloads DEVICE pointers (each demo_payload_bytes() bytes)
 *   n_payloads   must equal cfg.num_workers
 *   params       host array of n_tensors DEVICE pointers (fp32), updated in place
 * A record whose idx lies outside its chunk is skipped and DEMO_ERR_PAYLOAD becomes the sticky
 * device status.  Errors: INVALID_ARG, CUDA.
 */
demo_status demo_decode_apply(demo_ctx *ctx, const void *const *payloads, int32_t n_payloads,
                              float *const *params, void *cuda_stream);

/*
 * Parameter-server form of the server side (Algorithm 1: the server aggregates and reconstructs the
 * momentum and broadcasts sgn(m_t); every worker then applies x <- x - lr (sgn + weight_decay x)).
 *
 * demo_decode_signs -- S and R as in demo_decode_apply (same aggregation modes), but instead of updating
 * parameters writes sign(R) in {-1, 0, +1} as one int8 per parameter.
 *   signs_out    host array of n_tensors DEVICE pointers (int8, each shaped and ordered like its
 *                parameter tensor), overwritten; 16-byte aligned
 * Needs phi = DEMO_PHI_SIGN (INVALID_ARG otherwise).  2-D tensors run on the fast kernels where
 * demo_decode_apply does, everything else (and every tensor under a caller-supplied basis) on the dense
 * kernels.
 *
 * demo_apply_signs -- x <- x - lr (sign + weight_decay x) for every parameter, from such int8 tensors
 * (the broadcast's payload), with the context's current lr.
 *   signs        host array of n_tensors DEVICE pointers (int8), read-only
 *   params       host array of n_tensors DEVICE pointers (fp32), updated in place
 * The two calls together leave the parameters demo_decode_apply leaves: bit for bit where that runs on the
 * dense kernels, within one fp32 rounding of the update where it runs on the fast kernels (which fold
 * 1 - lr weight_decay into one factor).  Where the two forms run on different kernel families (a
 * caller-supplied basis at chunk size 64: tensor cores against CUDA cores) an element whose reconstructed
 * momentum is zero to rounding may get another sign, as between any two of the kernel families.  The small tables of these
 * two entry points are allocated on the first call of either (so the first call cannot be part of a
 * stream capture).  Errors: INVALID_ARG, ALLOC, CUDA.
 */
demo_status demo_decode_signs(demo_ctx *ctx, const void *const *payloads, int32_t n_payloads,
                              int8_t *const *signs_out, void *cuda_stream);
demo_status demo_apply_signs(demo_ctx *ctx, const int8_t *const *signs, float *const *params, void *cuda_stream);

/*
 * demo_step_host -- one whole optimizer step driven from HOST gradient buffers: for every worker
 * copy its gradients host->device into the caller's device staging tensors, compress, then decode
 * and apply, then (if host_payloads_out is not NULL) copy all W payloads device->host.  Everything
 * is ordered with cuda_stream; the host buffers must stay valid until the stream has drained
 * (use pinned memory for the copies to be asynchronous).  The gradient copies run on an internal
 * stream, created together with W events on the first call, so that the copy of worker w+1 overlaps
 * the compress of worker w; they start only after the work already queued on cuda_stream.
 *   host_grads         host array [W * n_tensors] of HOST pointers (worker-major)
 *   dev_grads          host array [W * n_tensors] of DEVICE pointers receiving the copies
 *   momentum           host array [W * n_tensors] of DEVICE pointers (fp32)
 *   payloads           host array [W] of DEVICE payload buffers
 *   params             host array [n_tensors] of DEVICE pointers (fp32)
 *   host_payloads_out  HOST buffer of W * demo_payload_bytes() bytes, or NULL
 * Errors: as demo_compress / demo_decode_apply.
 */
demo_status demo_step_host(demo_ctx *ctx, const void *const *host_grads, void *const *dev_grads,
                           float *const *momentum, void *const *payloads, float *const *params,
                           void *host_payloads_out, void *cuda_stream);

/*
 * demo_decode_apply_static -- the same decode + update as demo_decode_apply, for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is a deployment variant of the
 * server-side step, not another algorithm.)
 *
 * Who needs it: code running where cudaMalloc is off limits -- inside a memory pool that owns the
 * whole device, in a plug-in whose host forbids driver allocations after start-up, or on a stream
 * that must never hit an implicit synchronisation from an allocator.  demo_init allocates the
 * context's tables with cudaMalloc; this entry point needs no context and calls neither cudaMalloc,
 * cudaFree nor any allocating library routine.  The small tables the kernels read (DCT basis, tensor
 * table, the two pointer tables, a status word) live in one fixed array of DEMO_STATIC_SCRATCH_BYTES
 * bytes of device memory that every GPU loading this library holds until the process exits.
 *
 * Arguments are those of demo_init (cfg, tensors, n_tensors, cuda_device) plus those of
 * demo_decode_apply (payloads, n_payloads == cfg->num_workers, params, cuda_stream); cfg->beta and
 * cfg->grad_dtype are ignored.  Payloads and parameters are caller-owned DEVICE buffers, 16-byte
 * aligned; the pointer arrays are host memory read during the call.
 *
 * Limits (larger problems are rejected with DEMO_ERR_UNSUPPORTED before anything is enqueued):
 * n_tensors <= DEMO_STATIC_MAX_TENSORS, n_payloads <= DEMO_STATIC_MAX_WORKERS,
 * cfg->chunk <= DEMO_STATIC_MAX_CHUNK.
 *
 * Sharing: all calls in the process use the same array on a given device.  Each call rewrites the
 * tables and zeroes the status word in stream order, so consecutive calls on ONE stream are safe;
 * calls whose kernels may overlap on the GPU (different streams without ordering, several host
 * threads) race on the tables and must be serialised by the caller.  Records whose index lies outside
 * their chunk are skipped as in demo_decode_apply, but are not reported (there is no context to query).
 *
 * The first call on a device looks up the array's device address (a one-time set-up that should
 * happen before any stream capture begins).  Every call copies its tables from host memory that is
 * gone when the call returns, so the call must not be recorded into a CUDA graph: a stream that is
 * capturing is refused with DEMO_ERR_INVALID_ARG before anything is enqueued.  The 2-D and 1-D
 * tensors run through the generic decode kernels.  Errors: INVALID_ARG, SHAPE, K, UNSUPPORTED, CUDA.
 */
#define DEMO_STATIC_MAX_TENSORS 256
#define DEMO_STATIC_MAX_WORKERS 64
#define DEMO_STATIC_MAX_CHUNK 64
#define DEMO_STATIC_SCRATCH_BYTES (64 * 64 * 4 + 256 * 32 + 256 * 8 + 64 * 8 + 256)
demo_status demo_decode_apply_static(const demo_config *cfg, const demo_tensor_desc *tensors, int32_t n_tensors,
                                     const void *const *payloads, int32_t n_payloads, float *const *params,
                                     int32_t cuda_device, void *cuda_stream);

/* The learning rate is scheduled (eta_t in the update equation of Section 2.1): takes effect for
 * the next demo_decode_apply.  Errors: INVALID_ARG (null ctx, non-finite lr). */
demo_status demo_set_lr(demo_ctx *ctx, float lr);

/* Momentum-subtraction coefficient of Section 2.1 ("Momentum Subtraction as Error Feedback"):
 * demo_compress leaves m <- (beta*m + g) - alpha * IDCT(kept coefficients); the records always carry
 * the full coefficients.  Default 1 (the algorithm listings); 0 <= alpha <= 1.  Takes effect for the
 * next demo_compress.  Errors: INVALID_ARG. */
demo_status demo_set_alpha(demo_ctx *ctx, float alpha);

/* How demo_decode_apply combines the W payloads and which transform phi it applies (Section 2.1):
 *   aggregation  DEMO_AGG_SUM         S = sum_w Q^w                         (Algorithm 1; default)
 *                DEMO_AGG_MEAN        S = (1/W) sum_w Q^w                   (AvgAllGather)
 *                DEMO_AGG_COUNT_MEAN  S[i] = sum_w Q^w[i] / #{w : i sent},  0/0 = 0
 *                                     (appendix algorithm "Sparse Top-k Averaging")
 *   phi          DEMO_PHI_SIGN        x <- x - lr (sign(R) + wd x)          (Signum; default)
 *                DEMO_PHI_IDENTITY    x <- x - lr (R + wd x)                (SGD-style)
 * with R = IDCT(S).  Takes effect for the next demo_decode_apply.
 * Errors: INVALID_ARG; UNSUPPORTED (count-normalised mean with more than 65535 workers). */
typedef enum { DEMO_AGG_SUM = 0, DEMO_AGG_MEAN = 1, DEMO_AGG_COUNT_MEAN = 2 } demo_aggregation;
typedef enum { DEMO_PHI_SIGN = 0, DEMO_PHI_IDENTITY = 1 } demo_phi;
demo_status demo_set_decode_mode(demo_ctx *ctx, int32_t aggregation, int32_t phi);

/* Other orthonormal bases (Section 4.2, "Choice of Linear Projections": identity mapping, random
 * orthonormal projection).  The basis is an s x s row-major fp32 matrix P whose ROWS are the basis
 * vectors; it replaces the DCT matrix on both axes of a 2-D chunk (Q = P B P^T, inverse P^T Q P) and on
 * 1-D segments (q = P b).  While a caller-supplied basis is active the fast kernels (which hard-code the
 * DCT factorisation) are out: 2-D tensors at chunk size 64 run on tensor-core kernels (3xTF32, fp32
 * accuracy), everything else on the dense CUDA-core kernels; DEMO_PATH_GENERIC forces the latter.
 *
 * demo_set_basis: basis_host = HOST pointer to P, read during the call and not retained; NULL restores
 * the DCT.  The rows must be orthonormal to 1e-5 (INVALID_ARG otherwise).  The upload is enqueued on
 * cuda_stream, so the new basis applies to calls enqueued after it on that stream.
 *
 * demo_set_basis_gaussian: gauss_host = HOST pointer to an s x s row-major matrix of N(0,1) draws (the
 * paper seeds them with the step number so that all workers agree).  Its rows are orthonormalised in
 * order by the Gram-Schmidt process on the device (fp64, one small kernel) and the result becomes the
 * active basis.  Synchronises cuda_stream.  INVALID_ARG when a row has no component left (singular
 * matrix); the previous basis then stays in force.
 *
 * demo_get_basis: copies the active basis (DCT or caller-supplied) to basis_host_out (HOST, s*s floats)
 * and synchronises cuda_stream.
 * Errors: INVALID_ARG, CUDA. */
demo_status demo_set_basis(demo_ctx *ctx, const float *basis_host, void *cuda_stream);
demo_status demo_set_basis_gaussian(demo_ctx *ctx, const float *gauss_host, void *cuda_stream);
demo_status demo_get_basis(demo_ctx *ctx, float *basis_host_out, void *cuda_stream);

/* Self-test of the device-side failure path: enqueue a one-CTA kernel that waits, for at most
 * limit_cycles SM clock cycles (1 .. 2e9), on a barrier that nothing completes -- the situation a lost
 * tile copy would create -- using the same bounded wait as the production kernels.  The kernel records
 * DEMO_ERR_TIMEOUT in the sticky device status and returns; the context stays usable.  Nothing is
 * trapped, faulted or left spinning.  Errors: INVALID_ARG, CUDA. */
demo_status demo_selftest_bounded_wait(demo_ctx *ctx, int64_t limit_cycles, void *cuda_stream);

/* Select the kernel family (see demo_path).  Errors: INVALID_ARG. */
demo_status demo_set_path(demo_ctx *ctx, int32_t path);

/* Representation of the momentum tensors of 2-D parameters (opt-in; the paper keeps the momentum itself and
 * has no counterpart of this switch).  The chunk transform is linear and orthonormal, so the step of
 * Algorithm 1 can be carried out on the transformed momentum Qm = DCT(m) chunk by chunk:
 *     Q = beta * Qm + DCT(g);   records = top-k(Q);   Qm <- Q - alpha * Q_kept,
 * which yields the records of demo_compress up to fp32 rounding and needs one forward transform of the
 * gradient and no inverse transform.
 *   DEMO_MOMENTUM_SPATIAL (default): the buffers passed to demo_compress hold m.
 *   DEMO_MOMENTUM_DCT: for every 2-D tensor they hold, tile by tile, the TRANSPOSED coefficient tile of
 *     the chunk: element (64*k0 + r, 64*k1 + c) of the buffer is coefficient (c, r) of chunk (k0, k1) of
 *     DCT(m).  An all-zero buffer means m = 0 in both representations.  The momentum is recovered as
 *     m = IDCT(tile transposed) per chunk; 1-D tensors always hold m itself.
 * Only the s = 64 tile kernel with TMA tensor maps implements the second form: UNSUPPORTED for contexts
 * of demo_init_nd, for chunk != 64, or when the driver offers no tensor-map encoder; while it is on,
 * demo_compress (and demo_step_host, which calls it) returns UNSUPPORTED if a caller-supplied basis or
 * DEMO_PATH_GENERIC is active.  The caller converts or clears the buffers when switching; the library
 * never does.  Errors: INVALID_ARG, UNSUPPORTED. */
typedef enum demo_momentum_domain { DEMO_MOMENTUM_SPATIAL = 0, DEMO_MOMENTUM_DCT = 1 } demo_momentum_domain;
demo_status demo_set_momentum_domain(demo_ctx *ctx, int32_t domain);

/* Number of kernel launches this context has enqueued since demo_init (for accounting). */
int64_t demo_launch_count(const demo_ctx *ctx);

/* Synchronise cuda_stream and return (and clear) the sticky device status word: DEMO_OK,
 * DEMO_ERR_TIMEOUT or DEMO_ERR_PAYLOAD; DEMO_ERR_CUDA if the synchronisation itself failed. */
demo_status demo_device_status(demo_ctx *ctx, void *cuda_stream);

const char *demo_status_string(demo_status status);

/* Release the context's host and device memory.  NULL-safe.  Caller-owned tensors are untouched. */
void demo_free(demo_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* DEMO_H_ */
