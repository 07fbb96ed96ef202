// Internal declarations shared by the host library and the kernel translation units.
// Nothing here is part of the public ABI (see include/demo.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

// One payload record: flat index inside the chunk + fp32 coefficient (8 bytes, little-endian).
struct DemoRecord {
    int32_t idx;
    float val;
};

// One tensor of a work list.  A work list holds either all 2-D tensors or all 1-D tensors; chunk
// ids run over the list, row-major over each tensor's chunk grid (blocking operator, appendix
// B.1.2 of the paper).
struct DemoTensorEntry {
    long long chunk_begin;  // id of this tensor's first chunk inside the list
    long long rec_begin;    // index of this tensor's first record inside a payload
    int tensor;             // position in the caller's pointer arrays
    int n1;                 // row length in elements (2-D: shape[1]; 1-D: shape[0])
    int c1;                 // chunks per row of the chunk grid
    int k_eff;              // min(k, M)
};

struct DemoCompressArgs {
    const DemoTensorEntry *entries;  // device
    int n_entries;
    long long n_chunks;
    const void *const *g_ptrs;  // device array indexed by DemoTensorEntry::tensor
    float *const *m_ptrs;       // device array
    DemoRecord *payload;        // device, whole payload of this worker
    const float *C;             // device, s x s orthonormal DCT-II, C[u*s + n]
    float beta;
    float alpha;    // momentum-subtraction coefficient: m <- B - alpha * IDCT(kept)
    int grad_bf16;  // 1: gradients are bf16, 0: fp32
    int *status;    // device status word (sticky)
    // Optional TMA tensor maps (128-byte CUtensorMap objects in device memory, indexed like the
    // pointer arrays; box = one s x s tile).  NULL: tiles are staged row by row with 1-D bulk copies.
    const void *tmap_m;
    const void *tmap_g;
    // 1: the momentum tensors hold the chunk-wise DCT of the momentum (tiles transposed); only the s = 64 tile
    // kernel with tensor maps implements it
    int momentum_dct = 0;
};

struct DemoDecodeArgs {
    const DemoTensorEntry *entries;
    int n_entries;
    long long n_chunks;
    const DemoRecord *const *payloads;  // device array [W]
    int W;
    float *const *x_ptrs;  // device array
    const float *C;
    float lr;
    float wd;
    int *status;
    const void *tmap_x;  // optional tensor maps of the parameter tensors (see DemoCompressArgs)
    int agg;          // 0 sum, 1 mean over workers, 2 per-coordinate count-normalised mean (0/0 = 0)
    int phi;          // 0 sign, 1 identity
    float agg_scale;  // 1/W for the mean, else 1 (only the identity update sees it)
    // Parameter-server form: when not NULL, write sign(R) in {-1, 0, +1} per element to these int8 tensors
    // (device array indexed like x_ptrs) instead of updating the parameters.
    signed char *const *sign_ptrs = nullptr;
};

// Launchers (defined in the kernel translation units).  `s` is the chunk size, `two_d` selects
// s x s tiles (1) or length-s segments (0).  Return the CUDA error of the launch.
cudaError_t demo_launch_compress_generic(int s, int two_d, const DemoCompressArgs &a, int sm_count,
                                         cudaStream_t stream);
cudaError_t demo_launch_decode_generic(int s, int two_d, const DemoDecodeArgs &a, int sm_count,
                                       cudaStream_t stream);
// Fast-DCT kernels for 2-D tensors; `supported` tells whether chunk size s has one.
bool demo_fast_supported(int s);
cudaError_t demo_launch_compress_fast(int s, const DemoCompressArgs &a, int sm_count, cudaStream_t stream);
cudaError_t demo_launch_decode_fast(int s, const DemoDecodeArgs &a, int sm_count, cudaStream_t stream);
// s = 64 with TMA tensor maps (kernels_fast64.cu; cudaErrorNotSupported without them).
cudaError_t demo_launch_compress_fast64(const DemoCompressArgs &a, int sm_count, cudaStream_t stream);
// s = 128 (kernels_fast128.cu); need the TMA tensor maps (cudaErrorNotSupported without them).
cudaError_t demo_launch_compress_fast128(const DemoCompressArgs &a, int sm_count, cudaStream_t stream);
cudaError_t demo_launch_decode_fast128(const DemoDecodeArgs &a, int sm_count, cudaStream_t stream);

// Tensor-core kernels for 2-D tensors under a caller-supplied basis (kernels_tc.cu): tcgen05 MMAs with
// 3xTF32 splitting, chunk size 64 only.
bool demo_tc_supported(int s);
cudaError_t demo_launch_compress_tc(const DemoCompressArgs &a, int sm_count, cudaStream_t stream);
cudaError_t demo_launch_decode_tc(const DemoDecodeArgs &a, int sm_count, cudaStream_t stream);

// Self-test of the bounded wait (kernels_fast.cu): one CTA waits, for at most `limit_cycles`, on an
// mbarrier that nothing completes, records DEMO_DEV_TIMEOUT in *status and returns.
cudaError_t demo_launch_wait_selftest(int *status, long long limit_cycles, cudaStream_t stream);

// Gram-Schmidt process on the rows of the s x s matrix `gauss` (device, fp32) in fp64; writes the
// orthonormal rows to `basis` (device, fp32) and 1 to *flag when a row has no component left.
cudaError_t demo_launch_gram_schmidt(const float *gauss, float *basis, int *flag, int s, cudaStream_t stream);

// ---- tensors of any order with rectangular chunks (appendix of the paper: blocking operator and
// multilinear product; kernels_nd.cu) ---------------------------------------------------------------
constexpr int DEMO_ND_DIMS = 4;  // lower orders are padded on the left with axes of extent 1

struct DemoNdEntry {
    long long chunk_begin;           // id of this tensor's first chunk inside the work list
    long long chunk_end;             // chunk_begin + number of chunks of this tensor
    long long rec_begin;             // index of this tensor's first record inside a payload
    long long stride[DEMO_ND_DIMS];  // element stride of each axis of the (contiguous) tensor
    int tensor;                      // position in the caller's pointer arrays
    int k_eff;                       // min(k, M)
    int M;                           // elements per chunk
    int s[DEMO_ND_DIMS];             // chunk shape
    int c[DEMO_ND_DIMS];             // chunk grid
    unsigned inv[DEMO_ND_DIMS];      // ceil(2^32 / s[a]) for s[a] > 1 (division by multiplication), else 0
    int basis[DEMO_ND_DIMS];         // offset (floats, multiple of 4) of axis a's [C | C^T] inside the table
};

struct DemoNdCompressArgs {
    const DemoNdEntry *entries;  // device
    int n_entries;
    long long n_chunks;
    const void *const *g_ptrs;
    float *const *m_ptrs;
    DemoRecord *payload;
    const float *tables;  // device: per chunk extent s in use, C (s x s, C[u*s + n]) followed by C^T
    float beta, alpha;
    int grad_bf16;
    int max_M;  // largest chunk of the list (sizes the shared-memory buffers)
    int *status;
};

struct DemoNdDecodeArgs {
    const DemoNdEntry *entries;
    int n_entries;
    long long n_chunks;
    const DemoRecord *const *payloads;
    int W;
    float *const *x_ptrs;
    const float *tables;
    float lr, wd;
    int max_M;
    int *status;
    int agg, phi;
    float agg_scale;
    signed char *const *sign_ptrs = nullptr;  // see DemoDecodeArgs
};

// x <- x - lr (sign + wd x) from int8 signs, over every tensor of a context (kernels_generic.cu).
struct DemoFlatEntry {
    long long quad_begin;  // index of this tensor's first group of four elements in the launch
    long long n;           // elements
    int tensor;            // position in the pointer arrays
    int pad;
};
struct DemoApplySignsArgs {
    const DemoFlatEntry *entries;  // device
    int n_entries;
    long long n_quads;
    const signed char *const *sign_ptrs;  // device array
    float *const *x_ptrs;                 // device array
    float lr, wd;
};
cudaError_t demo_launch_apply_signs(const DemoApplySignsArgs &a, int sm_count, cudaStream_t stream);

cudaError_t demo_launch_compress_nd(const DemoNdCompressArgs &a, int sm_count, cudaStream_t stream);
cudaError_t demo_launch_decode_nd(const DemoNdDecodeArgs &a, int sm_count, cudaStream_t stream);

// Locate the tensor that owns chunk id c: the last entry with chunk_begin <= c.
__device__ __forceinline__ int demo_find_entry(const DemoTensorEntry *entries, int n, long long c)
{
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (entries[mid].chunk_begin <= c)
            lo = mid;
        else
            hi = mid - 1;
    }
    return lo;
}

// Status values written by kernels (match demo_status in include/demo.h).
#define DEMO_DEV_TIMEOUT 7
#define DEMO_DEV_PAYLOAD 8
