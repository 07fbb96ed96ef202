// Generic kernels of the DeMo optimizer transform: any chunk size s in {8,16,32,64,128}, 2-D tiles
// and 1-D segments, any k <= M.  One CTA works on one chunk at a time; the chunk stays in shared
// memory from the momentum update to the residual write-back, so HBM is touched once per operand.
// The chunk DCT here is the dense contraction with the precomputed basis (the paper's own cost
// model, Section 2.1 "Complexity Analysis"); the register-resident fast-DCT kernels for the common
// sizes live in kernels_fast.cu.  These kernels are the path for 1-D tensors, for s in {8,16,128}
// and the cross-check of the fast path.
#include <cuda_bf16.h>

#include "demo_internal.h"
#include "generic_common.cuh"

namespace {

// out[r][c] = sum_t L[r*lsr + t*lst] * R[t*rst + c*rsc]   (r < NR, c < NC, t < NT; out row-major)
template <int NR, int NC, int NT>
__device__ __forceinline__ void mm(float *__restrict__ out, const float *__restrict__ L, int lsr, int lst,
                                   const float *__restrict__ R, int rst, int rsc)
{
    constexpr int TR = (NR >= 4) ? 4 : 1;
    constexpr int TC = 4;
    constexpr int tiles_c = NC / TC;
    constexpr int n_tiles = (NR / TR) * tiles_c;
    for (int tile = threadIdx.x; tile < n_tiles; tile += GEN_THREADS) {
        const int r0 = (tile / tiles_c) * TR, c0 = (tile % tiles_c) * TC;
        float acc[TR][TC];
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < TC; ++j) acc[i][j] = 0.f;
#pragma unroll 4
        for (int t = 0; t < NT; ++t) {
            float l[TR], rr[TC];
#pragma unroll
            for (int i = 0; i < TR; ++i) l[i] = L[(r0 + i) * lsr + t * lst];
#pragma unroll
            for (int j = 0; j < TC; ++j) rr[j] = R[t * rst + (c0 + j) * rsc];
#pragma unroll
            for (int i = 0; i < TR; ++i)
#pragma unroll
                for (int j = 0; j < TC; ++j) acc[i][j] = fmaf(l[i], rr[j], acc[i][j]);
        }
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < TC; ++j) out[(r0 + i) * NC + c0 + j] = acc[i][j];
    }
}

// Forward chunk DCT: 2-D  Q = C B C^T,  1-D  q = C b.  Result in `q_out`, `tmp` is scratch.
template <int S, int ROWS>
__device__ __forceinline__ void forward_dct(const float *Bt, float *tmp, float *q_out, const float *C)
{
    if (ROWS > 1) {
        mm<ROWS, S, S>(tmp, Bt, S, 1, C, 1, S);  // tmp[i][v] = sum_j B[i][j] C[v][j]
        __syncthreads();
        mm<S, S, S>(q_out, C, S, 1, tmp, S, 1);  // Q[u][v] = sum_i C[u][i] tmp[i][v]
    } else {
        mm<ROWS, S, S>(q_out, Bt, S, 1, C, 1, S);
    }
    __syncthreads();
}

// Inverse chunk DCT: 2-D  R = C^T Q C,  1-D  r = C^T q.  Result in `r_out`, `tmp` is scratch.
template <int S, int ROWS>
__device__ __forceinline__ void inverse_dct(const float *Qt, float *tmp, float *r_out, const float *C)
{
    if (ROWS > 1) {
        mm<ROWS, S, S>(tmp, Qt, S, 1, C, S, 1);   // tmp[u][j] = sum_v Q[u][v] C[v][j]
        __syncthreads();
        mm<S, S, S>(r_out, C, 1, S, tmp, S, 1);   // R[i][j] = sum_u C[u][i] tmp[u][j]
    } else {
        mm<ROWS, S, S>(r_out, Qt, S, 1, C, S, 1);
    }
    __syncthreads();
}

template <int S, int ROWS>
__global__ void __launch_bounds__(GEN_THREADS) compress_generic_kernel(DemoCompressArgs a)
{
    constexpr int M = ROWS * S;
    extern __shared__ float smem[];
    float *Bt = smem;
    float *X1 = Bt + M;
    float *X2 = X1 + M;
    unsigned *hist = reinterpret_cast<unsigned *>(X2 + M);  // [256]
    unsigned *warp_tot = hist + 256;                        // [8]
    unsigned *s_state = warp_tot + 8;                       // [2]
    const int tid = threadIdx.x;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        const DemoTensorEntry te = a.entries[demo_find_entry(a.entries, a.n_entries, c)];
        const long long lc = c - te.chunk_begin;
        const long long k0 = lc / te.c1;
        const int k1 = (int)(lc - k0 * te.c1);
        const size_t base = (size_t)k0 * ROWS * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ m = a.m_ptrs[te.tensor];
        const void *g = a.g_ptrs[te.tensor];
        const int k_eff = te.k_eff;

        // momentum update  B = beta*m + g  on the chunk (Algorithm 1, worker side)
        for (int i = tid; i < M; i += GEN_THREADS) {
            const int r = i / S, j = i - r * S;
            const size_t off = base + (size_t)r * te.n1 + j;
            const float gv = a.grad_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(g)[off])
                                         : reinterpret_cast<const float *>(g)[off];
            Bt[i] = fmaf(a.beta, m[off], gv);
        }
        __syncthreads();

        float *Q = (ROWS > 1) ? X2 : X1;   // coefficients
        float *O = (ROWS > 1) ? X1 : X2;   // the other buffer
        forward_dct<S, ROWS>(Bt, X1, Q, a.C);

        // top-k: threshold by radix select, then index-ordered compaction into the payload
        unsigned thr, need_eq;
        radix_select(Q, M, k_eff, hist, s_state, &thr, &need_eq);
        constexpr int PER = (M + GEN_THREADS - 1) / GEN_THREADS;
        const int start = tid * PER;
        unsigned gt = 0, eq = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int i = start + j;
            if (i < M) {
                const unsigned key = mag_key(Q[i]);
                gt += key > thr;
                eq += key == thr;
            }
        }
        const unsigned before = block_exclusive_scan(gt | (eq << 16), warp_tot);
        unsigned gb = before & 0xffffu, eb = before >> 16;
        DemoRecord *rec = a.payload + te.rec_begin + lc * (long long)k_eff;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int i = start + j;
            if (i < M) {
                const float v = Q[i];
                const unsigned key = mag_key(v);
                bool sel = false;
                unsigned pos = 0;
                if (key > thr) {
                    pos = gb + min(eb, need_eq);
                    ++gb;
                    sel = true;
                } else if (key == thr) {
                    if (eb < need_eq) {
                        pos = gb + eb;
                        sel = true;
                    }
                    ++eb;
                }
                if (sel) {
                    DemoRecord r;
                    r.idx = i;
                    r.val = v;
                    rec[pos] = r;
                }
                O[i] = sel ? a.alpha * v : 0.f;  // the residual removes alpha times the kept part
            }
        }
        __syncthreads();

        // momentum subtraction  m <- B - IDCT(kept coefficients)
        float *R = (ROWS > 1) ? O : Q;
        inverse_dct<S, ROWS>(O, Q, R, a.C);
        for (int i = tid; i < M; i += GEN_THREADS) {
            const int r = i / S, j = i - r * S;
            m[base + (size_t)r * te.n1 + j] = Bt[i] - R[i];
        }
        __syncthreads();
    }
}

template <int S, int ROWS>
__global__ void __launch_bounds__(GEN_THREADS) decode_generic_kernel(DemoDecodeArgs a)
{
    constexpr int M = ROWS * S;
    extern __shared__ float smem[];
    float *St = smem;
    float *X1 = St + M;
    unsigned short *Cn = reinterpret_cast<unsigned short *>(X1 + M);  // [M] senders per coordinate (agg == 2 only)
    const int tid = threadIdx.x;
    const bool counts = a.agg == 2;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        const DemoTensorEntry te = a.entries[demo_find_entry(a.entries, a.n_entries, c)];
        const long long lc = c - te.chunk_begin;
        const long long k0 = lc / te.c1;
        const int k1 = (int)(lc - k0 * te.c1);
        const size_t base = (size_t)k0 * ROWS * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ x = a.x_ptrs[te.tensor];
        const int k_eff = te.k_eff;
        const long long rec_off = te.rec_begin + lc * (long long)k_eff;

        for (int i = tid; i < M; i += GEN_THREADS) {
            St[i] = 0.f;
            if (counts) Cn[i] = 0;
        }
        __syncthreads();
        // aggregate: S = sum over workers, in worker order (Decompress&Aggregate); indices are
        // unique inside one worker's chunk, so a barrier per worker fixes the summation order
        for (int w = 0; w < a.W; ++w) {
            const DemoRecord *rec = a.payloads[w] + rec_off;
            for (int i = tid; i < k_eff; i += GEN_THREADS) {
                const DemoRecord r = rec[i];
                if ((unsigned)r.idx < (unsigned)M) {
                    St[r.idx] += r.val;
                    if (counts) Cn[r.idx] += 1;
                } else {
                    atomicMax(a.status, DEMO_DEV_PAYLOAD);
                }
            }
            __syncthreads();
        }
        if (counts) {  // Sparse Top-k Averaging: sum / number of senders, 0/0 = 0
            for (int i = tid; i < M; i += GEN_THREADS) {
                const unsigned short n = Cn[i];
                if (n > 1) St[i] = St[i] / (float)n;
            }
            __syncthreads();
        }
        float *R = (ROWS > 1) ? St : X1;
        inverse_dct<S, ROWS>(St, X1, R, a.C);
        // x <- x - lr * (sign(R) + wd * x), sign(0) = 0
        for (int i = tid; i < M; i += GEN_THREADS) {
            const int r = i / S, j = i - r * S;
            const size_t off = base + (size_t)r * te.n1 + j;
            const float rv = R[i];
            if (a.sign_ptrs) {  // parameter-server form: hand out sign(R), the workers apply it
                a.sign_ptrs[te.tensor][off] = (signed char)((rv > 0.f) - (rv < 0.f));
                continue;
            }
            const float sg = a.phi ? rv * a.agg_scale : (float)((rv > 0.f) - (rv < 0.f));
            const float xv = x[off];
            x[off] = fmaf(-a.lr, fmaf(a.wd, xv, sg), xv);
        }
        __syncthreads();
    }
}

// x <- x - lr (sign + wd x) with the signs a parameter server handed out (Algorithm 1, last two lines).
// One thread per group of four consecutive elements of a tensor; same arithmetic as the decode kernels.
__global__ void __launch_bounds__(GEN_THREADS) apply_signs_kernel(DemoApplySignsArgs a)
{
    for (long long q = (long long)blockIdx.x * GEN_THREADS + threadIdx.x; q < a.n_quads;
         q += (long long)gridDim.x * GEN_THREADS) {
        int lo = 0, hi = a.n_entries - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (a.entries[mid].quad_begin <= q)
                lo = mid;
            else
                hi = mid - 1;
        }
        const DemoFlatEntry e = a.entries[lo];
        const long long i0 = (q - e.quad_begin) * 4;
        float *__restrict__ x = a.x_ptrs[e.tensor];
        const signed char *__restrict__ sg = a.sign_ptrs[e.tensor];
        if (i0 + 4 <= e.n) {  // tensors start 16-byte aligned, so groups of four are aligned too
            float4 xv = *reinterpret_cast<const float4 *>(x + i0);
            const char4 s4 = *reinterpret_cast<const char4 *>(sg + i0);
            xv.x = fmaf(-a.lr, fmaf(a.wd, xv.x, (float)s4.x), xv.x);
            xv.y = fmaf(-a.lr, fmaf(a.wd, xv.y, (float)s4.y), xv.y);
            xv.z = fmaf(-a.lr, fmaf(a.wd, xv.z, (float)s4.z), xv.z);
            xv.w = fmaf(-a.lr, fmaf(a.wd, xv.w, (float)s4.w), xv.w);
            *reinterpret_cast<float4 *>(x + i0) = xv;
        } else {
            for (long long i = i0; i < e.n; ++i) {
                const float xv = x[i];
                x[i] = fmaf(-a.lr, fmaf(a.wd, xv, (float)sg[i]), xv);
            }
        }
    }
}

template <int S>
cudaError_t compress_dispatch(int two_d, const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    const size_t extra = (256 + 8 + 2) * sizeof(unsigned);
    if (two_d)
        return launch_persistent(compress_generic_kernel<S, S>, 3 * S * S * sizeof(float) + extra, a.n_chunks,
                                 sm_count, stream, &a);
    return launch_persistent(compress_generic_kernel<S, 1>, 3 * S * sizeof(float) + extra, a.n_chunks, sm_count,
                             stream, &a);
}

template <int S>
cudaError_t decode_dispatch(int two_d, const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    if (two_d)
        return launch_persistent(decode_generic_kernel<S, S>, 2 * S * S * sizeof(float) + S * S * 2, a.n_chunks, sm_count,
                                 stream, &a);
    return launch_persistent(decode_generic_kernel<S, 1>, 2 * S * sizeof(float) + S * 2, a.n_chunks, sm_count, stream, &a);
}

}  // namespace

cudaError_t demo_launch_compress_generic(int s, int two_d, const DemoCompressArgs &a, int sm_count,
                                         cudaStream_t stream)
{
    switch (s) {
        case 8: return compress_dispatch<8>(two_d, a, sm_count, stream);
        case 16: return compress_dispatch<16>(two_d, a, sm_count, stream);
        case 32: return compress_dispatch<32>(two_d, a, sm_count, stream);
        case 64: return compress_dispatch<64>(two_d, a, sm_count, stream);
        case 128: return compress_dispatch<128>(two_d, a, sm_count, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t demo_launch_apply_signs(const DemoApplySignsArgs &a, int sm_count, cudaStream_t stream)
{
    if (a.n_quads <= 0) return cudaSuccess;
    long long grid = (a.n_quads + GEN_THREADS - 1) / GEN_THREADS;
    const long long cap = (long long)sm_count * 8;
    if (grid > cap) grid = cap;
    apply_signs_kernel<<<(unsigned)grid, GEN_THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t demo_launch_decode_generic(int s, int two_d, const DemoDecodeArgs &a, int sm_count,
                                       cudaStream_t stream)
{
    switch (s) {
        case 8: return decode_dispatch<8>(two_d, a, sm_count, stream);
        case 16: return decode_dispatch<16>(two_d, a, sm_count, stream);
        case 32: return decode_dispatch<32>(two_d, a, sm_count, stream);
        case 64: return decode_dispatch<64>(two_d, a, sm_count, stream);
        case 128: return decode_dispatch<128>(two_d, a, sm_count, stream);
        default: return cudaErrorInvalidValue;
    }
}

// =================================================================================================
// Random orthonormal basis (Section 4.2, "Choice of Linear Projections"): Gram-Schmidt process on the
// rows of a Gaussian matrix, in fp64, one CTA.  Right-looking order: once row j is final its component
// is removed from every later row, so each row loses its components along rows 0..j-1 one after the
// other -- the same operations as the row-by-row statement of the process.
// =================================================================================================
constexpr int GS_THREADS = 1024;

__global__ void __launch_bounds__(GS_THREADS) gram_schmidt_kernel(const float *__restrict__ gauss,
                                                                  float *__restrict__ basis, int *flag, int s)
{
    extern __shared__ double gs_A[];  // [s][s + 1]
    __shared__ double scale[128];     // squared length of each input row
    __shared__ double inv_len;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int WARPS = GS_THREADS / 32;
    const int ld = s + 1;
    for (int i = tid; i < s * s; i += GS_THREADS) gs_A[(i / s) * ld + (i % s)] = (double)gauss[i];
    __syncthreads();
    for (int r = warp; r < s; r += WARPS) {
        double acc = 0.0;
        for (int n = lane; n < s; n += 32) acc += gs_A[r * ld + n] * gs_A[r * ld + n];
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
        if (lane == 0) scale[r] = acc;
    }
    __syncthreads();
    bool bad = false;
    for (int j = 0; j < s; ++j) {
        if (warp == 0) {
            double acc = 0.0;
            for (int n = lane; n < s; n += 32) acc += gs_A[j * ld + n] * gs_A[j * ld + n];
            for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
            if (lane == 0) inv_len = (acc > 1e-24 * scale[j]) ? 1.0 / sqrt(acc) : 0.0;
        }
        __syncthreads();
        const double inv = inv_len;
        if (inv == 0.0) {
            bad = true;
            break;
        }
        double p[4];  // s <= 128: at most 4 entries of row j per lane
#pragma unroll
        for (int t = 0; t < 4; ++t) p[t] = (lane + 32 * t < s) ? gs_A[j * ld + lane + 32 * t] * inv : 0.0;
        for (int r = j + 1 + warp; r < s; r += WARPS) {
            double dot = 0.0;
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (lane + 32 * t < s) dot += gs_A[r * ld + lane + 32 * t] * p[t];
            for (int d = 16; d > 0; d >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, d);
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (lane + 32 * t < s) gs_A[r * ld + lane + 32 * t] -= dot * p[t];
        }
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (lane + 32 * t < s) gs_A[j * ld + lane + 32 * t] = p[t];
        }
    }
    __syncthreads();
    if (bad) {
        if (tid == 0) *flag = 1;
        return;
    }
    for (int i = tid; i < s * s; i += GS_THREADS) basis[i] = (float)gs_A[(i / s) * ld + (i % s)];
}

cudaError_t demo_launch_gram_schmidt(const float *gauss, float *basis, int *flag, int s, cudaStream_t stream)
{
    if (s < 1 || s > 128) return cudaErrorInvalidValue;
    const size_t smem = sizeof(double) * (size_t)s * (s + 1);
    cudaError_t err =
        cudaFuncSetAttribute(gram_schmidt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    gram_schmidt_kernel<<<1, GS_THREADS, smem, stream>>>(gauss, basis, flag, s);
    return cudaGetLastError();
}

// =================================================================================================
// demo_decode_apply_static: the decode + update step for callers that must not allocate.
//
// The generic decode kernels above read four small tables from global memory besides the caller's
// payloads and parameters: the DCT basis, the tensor table, the two pointer tables and a status
// word.  A context built by demo_init gets them from cudaMalloc; this entry point keeps them in the
// fixed array below instead, so it never allocates -- at the price of hard limits on the problem
// size and of one array shared by every call in the process.
// =================================================================================================
#include <cmath>
#include <cstring>
#include <mutex>

#include "../../include/demo.h"

namespace {

constexpr int STATIC_MAX_TENSORS = DEMO_STATIC_MAX_TENSORS;
constexpr int STATIC_MAX_WORKERS = DEMO_STATIC_MAX_WORKERS;
constexpr int STATIC_MAX_CHUNK = DEMO_STATIC_MAX_CHUNK;

// layout of the scratch array (byte offsets, all multiples of 256)
constexpr size_t OFF_BASIS = 0;                                                                   // s*s floats
constexpr size_t OFF_ENTRIES = OFF_BASIS + sizeof(float) * STATIC_MAX_CHUNK * STATIC_MAX_CHUNK;   // tensor table
constexpr size_t OFF_XPTRS = OFF_ENTRIES + sizeof(DemoTensorEntry) * STATIC_MAX_TENSORS;          // float*[T]
constexpr size_t OFF_PPTRS = OFF_XPTRS + sizeof(void *) * STATIC_MAX_TENSORS;                     // record*[W]
constexpr size_t OFF_STATUS = OFF_PPTRS + sizeof(void *) * STATIC_MAX_WORKERS;                    // int
constexpr size_t STATIC_SCRATCH_BYTES = OFF_STATUS + 256;

static_assert(STATIC_SCRATCH_BYTES == DEMO_STATIC_SCRATCH_BYTES, "header and layout disagree");

}  // namespace

// Device-resident scratch.  In host code this name is only a handle for cudaGetSymbolAddress; the
// device address is looked up once per device and passed to the kernels like any other pointer.
static __device__ __align__(256) unsigned char demo_static_scratch[DEMO_STATIC_SCRATCH_BYTES];

namespace {

constexpr int STATIC_MAX_DEVICES = 64;
std::mutex g_static_mutex;
unsigned char *g_static_base[STATIC_MAX_DEVICES];  // device address of the scratch, per device (0 = not set up)

}  // namespace

extern "C" demo_status demo_decode_apply_static(const demo_config *cfg, const demo_tensor_desc *tensors,
                                                int32_t n_tensors, const void *const *payloads, int32_t n_payloads,
                                                float *const *params, int32_t cuda_device, void *cuda_stream)
{
    if (!cfg || !tensors || !payloads || !params || n_tensors < 1 || cuda_device < 0) return DEMO_ERR_INVALID_ARG;
    if (cuda_device >= STATIC_MAX_DEVICES) return DEMO_ERR_UNSUPPORTED;
    if (n_payloads < 1 || n_payloads != cfg->num_workers) return DEMO_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->lr) || !std::isfinite(cfg->weight_decay)) return DEMO_ERR_INVALID_ARG;
    const int s = cfg->chunk;
    if (!(s == 8 || s == 16 || s == 32 || s == 64 || s == 128)) return DEMO_ERR_UNSUPPORTED;
    // the fixed scratch bounds the problem: reject anything larger instead of overrunning it
    if (s > STATIC_MAX_CHUNK || n_tensors > STATIC_MAX_TENSORS || n_payloads > STATIC_MAX_WORKERS)
        return DEMO_ERR_UNSUPPORTED;
    if (cfg->topk < 1 || (long long)cfg->topk > (long long)s * s) return DEMO_ERR_K;
    for (int t = 0; t < n_tensors; ++t) {
        const demo_tensor_desc &d = tensors[t];
        if (d.ndim != 1 && d.ndim != 2) return DEMO_ERR_SHAPE;
        for (int ax = 0; ax < d.ndim; ++ax)
            if (d.shape[ax] < s || d.shape[ax] % s != 0 || d.shape[ax] > (1LL << 31) - 1) return DEMO_ERR_SHAPE;
        if (!params[t] || (reinterpret_cast<uintptr_t>(params[t]) & 15u)) return DEMO_ERR_INVALID_ARG;
    }
    for (int w = 0; w < n_payloads; ++w)
        if (!payloads[w] || (reinterpret_cast<uintptr_t>(payloads[w]) & 15u)) return DEMO_ERR_INVALID_ARG;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    if (prev != cuda_device && cudaSetDevice(cuda_device) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    demo_status result = DEMO_OK;
    do {
        // The tables are copied from host memory that is gone when this call returns (a stack frame, the
        // caller's pointer arrays).  Recorded into a CUDA graph those copies would be replayed from dead
        // memory, so a stream that is capturing is refused before anything is enqueued.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            result = DEMO_ERR_INVALID_ARG;
            break;
        }
        // one-time set-up per device, with that device current: translate the symbol into a device address
        unsigned char *base = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_static_mutex);
            if (!g_static_base[cuda_device]) {
                void *p = nullptr;
                if (cudaGetSymbolAddress(&p, demo_static_scratch) != cudaSuccess || !p) {
                    cudaGetLastError();
                    result = DEMO_ERR_CUDA;
                    break;
                }
                g_static_base[cuda_device] = static_cast<unsigned char *>(p);
            }
            base = g_static_base[cuda_device];
        }
        int sm_count = 0;
        if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, cuda_device) != cudaSuccess) {
            result = DEMO_ERR_CUDA;
            break;
        }

        // host-side images of the tables (fixed-size, on the stack / in static storage: no heap)
        static thread_local float h_basis[STATIC_MAX_CHUNK * STATIC_MAX_CHUNK];
        DemoTensorEntry h_entries[STATIC_MAX_TENSORS];  // 2-D tensors first, then 1-D tensors
        int n2d = 0, n1d = 0;
        long long chunks2d = 0, chunks1d = 0;
        {
            const double pi = 3.141592653589793238462643383279502884;
            for (int u = 0; u < s; ++u)
                for (int n = 0; n < s; ++n) {
                    const double au = (u == 0) ? std::sqrt(1.0 / s) : std::sqrt(2.0 / s);
                    h_basis[(size_t)u * s + n] = (float)(au * std::cos(pi * (2.0 * n + 1.0) * u / (2.0 * s)));
                }
            for (int t = 0; t < n_tensors; ++t) n2d += tensors[t].ndim == 2;
            int i2 = 0, i1 = n2d;
            long long rec = 0;
            for (int t = 0; t < n_tensors; ++t) {
                const demo_tensor_desc &d = tensors[t];
                const bool two = d.ndim == 2;
                const long long n1 = two ? d.shape[1] : d.shape[0];
                const long long c0 = two ? d.shape[0] / s : 1, c1 = n1 / s;
                const long long M = two ? (long long)s * s : s;
                DemoTensorEntry e;
                e.tensor = t;
                e.n1 = (int)n1;
                e.c1 = (int)c1;
                e.k_eff = (int)(cfg->topk < M ? cfg->topk : M);
                e.rec_begin = rec;
                e.chunk_begin = two ? chunks2d : chunks1d;
                (two ? chunks2d : chunks1d) += c0 * c1;
                h_entries[two ? i2++ : i1++] = e;
                rec += c0 * c1 * e.k_eff;
            }
            n1d = n_tensors - n2d;
        }

        bool ok = true;
        ok = ok && cudaMemcpyAsync(base + OFF_BASIS, h_basis, sizeof(float) * (size_t)s * s, cudaMemcpyHostToDevice,
                                   stream) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(base + OFF_ENTRIES, h_entries, sizeof(DemoTensorEntry) * (size_t)n_tensors,
                                   cudaMemcpyHostToDevice, stream) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(base + OFF_XPTRS, params, sizeof(void *) * (size_t)n_tensors, cudaMemcpyHostToDevice,
                                   stream) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(base + OFF_PPTRS, payloads, sizeof(void *) * (size_t)n_payloads,
                                   cudaMemcpyHostToDevice, stream) == cudaSuccess;
        // the array keeps the previous call's contents: the status word must start at zero
        ok = ok && cudaMemsetAsync(base + OFF_STATUS, 0, sizeof(int), stream) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            result = DEMO_ERR_CUDA;
            break;
        }

        DemoDecodeArgs a;
        a.payloads = reinterpret_cast<const DemoRecord *const *>(base + OFF_PPTRS);
        a.W = n_payloads;
        a.x_ptrs = reinterpret_cast<float *const *>(base + OFF_XPTRS);
        a.C = reinterpret_cast<const float *>(base + OFF_BASIS);
        a.lr = cfg->lr;
        a.wd = cfg->weight_decay;
        a.status = reinterpret_cast<int *>(base + OFF_STATUS);
        a.tmap_x = nullptr;
        a.agg = 0;
        a.phi = 0;
        a.agg_scale = 1.f;
        cudaError_t err = cudaSuccess;
        if (n2d) {
            a.entries = reinterpret_cast<const DemoTensorEntry *>(base + OFF_ENTRIES);
            a.n_entries = n2d;
            a.n_chunks = chunks2d;
            err = demo_launch_decode_generic(s, 1, a, sm_count, stream);
        }
        if (err == cudaSuccess && n1d) {
            a.entries = reinterpret_cast<const DemoTensorEntry *>(base + OFF_ENTRIES) + n2d;
            a.n_entries = n1d;
            a.n_chunks = chunks1d;
            err = demo_launch_decode_generic(s, 0, a, sm_count, stream);
        }
        if (err != cudaSuccess) {
            cudaGetLastError();
            result = DEMO_ERR_CUDA;
        }
    } while (false);
    if (prev >= 0 && prev != cuda_device) cudaSetDevice(prev);
    return result;
}
