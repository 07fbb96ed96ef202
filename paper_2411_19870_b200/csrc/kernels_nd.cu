// Kernels for tensors of any order (up to DEMO_ND_DIMS axes) cut into rectangular chunks
// s_0 x ... x s_{d-1}: the general statement of the method in the paper's appendix ("Multilinear
// Transforms and Chunk-wise Tensor Blocking").  The chunk transform is the multilinear product
// T(B; C_0, ..., C_{d-1}) with the DCT matrix of dimension s_a on axis a, applied one axis after the
// other as dense contractions on the CUDA cores; chunk extents are run-time values.  One CTA works on
// one chunk at a time and keeps it in shared memory from the momentum update to the residual
// write-back, so HBM is touched once per operand, as in the kernels for square chunks.  Selection,
// record layout and update are those of kernels_generic.cu.
#include <cuda_bf16.h>

#include "demo_internal.h"
#include "generic_common.cuh"

namespace {

// Last entry with chunk_begin <= c.
__device__ __forceinline__ int find_nd_entry(const DemoNdEntry *entries, int n, long long c)
{
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (entries[mid].chunk_begin <= c)
            lo = mid;
        else
            hi = mid - 1;
    }
    return lo;
}

// Element offset of the chunk's first element: chunk id -> (k_0..k_3) row-major over the chunk grid,
// offset = sum_a k_a s_a stride_a (blocking operator).
__device__ __forceinline__ size_t chunk_base(const DemoNdEntry &e, long long lc)
{
    size_t base = 0;
#pragma unroll
    for (int a = DEMO_ND_DIMS - 1; a >= 0; --a) {
        const long long k = lc % e.c[a];
        lc /= e.c[a];
        base += (size_t)k * (size_t)e.s[a] * (size_t)e.stride[a];
    }
    return base;
}

// Offset of element i (row-major inside the chunk) relative to the chunk's first element.
__device__ __forceinline__ size_t elem_offset(const DemoNdEntry &e, int i)
{
    size_t off = 0;
#pragma unroll
    for (int a = DEMO_ND_DIMS - 1; a >= 0; --a) {
        const int j = i % e.s[a];
        i /= e.s[a];
        off += (size_t)j * (size_t)e.stride[a];
    }
    return off;
}

// One axis of the multilinear product on a chunk in shared memory viewed as [outer][s][inner]:
//   forward  dst[o][u][i] = sum_n P[u][n] src[o][n][i]
//   inverse  dst[o][n][i] = sum_u P[u][n] src[o][u][i]
// Each thread produces TU outputs that share their inputs.
template <int TU>
__device__ __forceinline__ void axis_pass(float *__restrict__ dst, const float *__restrict__ src,
                                          const float *__restrict__ P, int s, int inner, int M, bool inverse)
{
    const int p_out = inverse ? 1 : s;  // step in P from one output to the next
    const int p_in = inverse ? s : 1;   // step in P along the contracted index
    const int groups = s / TU;
    const int items = M / TU;
    for (int it = threadIdx.x; it < items; it += GEN_THREADS) {
        const int i = it % inner;
        const int t = it / inner;
        const int ub = (t % groups) * TU;
        const int o = t / groups;
        const float *sp = src + (size_t)o * s * inner + i;
        const float *pp = P + ub * p_out;
        float acc[TU];
#pragma unroll
        for (int q = 0; q < TU; ++q) acc[q] = 0.f;
        for (int n = 0; n < s; ++n) {
            const float v = sp[n * inner];
#pragma unroll
            for (int q = 0; q < TU; ++q) acc[q] = fmaf(__ldg(pp + q * p_out + n * p_in), v, acc[q]);
        }
        float *dp = dst + (size_t)o * s * inner + (size_t)ub * inner + i;
#pragma unroll
        for (int q = 0; q < TU; ++q) dp[q * inner] = acc[q];
    }
}

// All axes in turn, ping-pong between `a` and `b` (src may be one of them or a third buffer, which is
// then left intact).  Returns where the result is; src itself when every extent is 1.
__device__ __forceinline__ float *transform_chunk(float *src, float *a, float *b, const DemoNdEntry &e,
                                                  const float *tables, bool inverse)
{
    float *cur = src;
    int inner = e.M;
    for (int ax = 0; ax < DEMO_ND_DIMS; ++ax) {
        const int s = e.s[ax];
        inner /= s;
        if (s == 1) continue;
        float *dst = (cur == a) ? b : a;
        if ((s & 3) == 0)
            axis_pass<4>(dst, cur, tables + e.basis[ax], s, inner, e.M, inverse);
        else
            axis_pass<1>(dst, cur, tables + e.basis[ax], s, inner, e.M, inverse);
        __syncthreads();
        cur = dst;
    }
    return cur;
}

__global__ void __launch_bounds__(GEN_THREADS) compress_nd_kernel(DemoNdCompressArgs a)
{
    extern __shared__ float smem[];
    float *Bt = smem;
    float *X1 = Bt + a.max_M;
    float *X2 = X1 + a.max_M;
    unsigned *hist = reinterpret_cast<unsigned *>(X2 + a.max_M);  // [256]
    unsigned *warp_tot = hist + 256;                              // [8]
    unsigned *s_state = warp_tot + 8;                             // [2]
    const int tid = threadIdx.x;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        const DemoNdEntry e = a.entries[find_nd_entry(a.entries, a.n_entries, c)];
        const long long lc = c - e.chunk_begin;
        const size_t base = chunk_base(e, lc);
        float *__restrict__ m = a.m_ptrs[e.tensor];
        const void *g = a.g_ptrs[e.tensor];
        const int M = e.M, k_eff = e.k_eff;

        // momentum update  B = beta*m + g  on the chunk (Algorithm 1, worker side)
        for (int i = tid; i < M; i += GEN_THREADS) {
            const size_t off = base + elem_offset(e, i);
            const float gv = a.grad_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(g)[off])
                                         : reinterpret_cast<const float *>(g)[off];
            Bt[i] = fmaf(a.beta, m[off], gv);
        }
        __syncthreads();

        float *Q = transform_chunk(Bt, X1, X2, e, a.tables, false);  // Q = T(B; C_0, ..., C_{d-1})
        float *O = (Q == X1) ? X2 : X1;

        // top-k: threshold by radix select, then index-ordered compaction into the payload
        unsigned thr, need_eq;
        radix_select(Q, M, k_eff, hist, s_state, &thr, &need_eq);
        const int per = (M + GEN_THREADS - 1) / GEN_THREADS;
        const int start = tid * per;
        const int stop = min(M, start + per);
        unsigned gt = 0, eq = 0;
        for (int i = start; i < stop; ++i) {
            const unsigned key = mag_key(Q[i]);
            gt += key > thr;
            eq += key == thr;
        }
        const unsigned before = block_exclusive_scan(gt | (eq << 16), warp_tot);
        unsigned gb = before & 0xffffu, eb = before >> 16;
        DemoRecord *rec = a.payload + e.rec_begin + lc * (long long)k_eff;
        for (int i = start; i < stop; ++i) {
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
        __syncthreads();

        // momentum subtraction  m <- B - alpha * T(kept; C_0^T, ..., C_{d-1}^T)
        float *spare = (O == X1) ? X2 : X1;
        const float *R = transform_chunk(O, spare, O, e, a.tables, true);
        for (int i = tid; i < M; i += GEN_THREADS) m[base + elem_offset(e, i)] = Bt[i] - R[i];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(GEN_THREADS) decode_nd_kernel(DemoNdDecodeArgs a)
{
    extern __shared__ float smem[];
    float *St = smem;
    float *X1 = St + a.max_M;
    unsigned short *Cn = reinterpret_cast<unsigned short *>(X1 + a.max_M);  // senders per coordinate (agg == 2)
    const int tid = threadIdx.x;
    const bool counts = a.agg == 2;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        const DemoNdEntry e = a.entries[find_nd_entry(a.entries, a.n_entries, c)];
        const long long lc = c - e.chunk_begin;
        const size_t base = chunk_base(e, lc);
        float *__restrict__ x = a.x_ptrs[e.tensor];
        const int M = e.M, k_eff = e.k_eff;
        const long long rec_off = e.rec_begin + lc * (long long)k_eff;

        for (int i = tid; i < M; i += GEN_THREADS) {
            St[i] = 0.f;
            if (counts) Cn[i] = 0;
        }
        __syncthreads();
        // S = sum over workers, in worker order; indices are unique inside one worker's chunk, so a
        // barrier per worker fixes the summation order
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
        const float *R = transform_chunk(St, X1, St, e, a.tables, true);
        // x <- x - lr * (phi(R) + wd * x), sign(0) = 0
        for (int i = tid; i < M; i += GEN_THREADS) {
            const size_t off = base + elem_offset(e, i);
            const float rv = R[i];
            const float sg = a.phi ? rv * a.agg_scale : (float)((rv > 0.f) - (rv < 0.f));
            const float xv = x[off];
            x[off] = fmaf(-a.lr, fmaf(a.wd, xv, sg), xv);
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t demo_launch_compress_nd(const DemoNdCompressArgs &a, int sm_count, cudaStream_t stream)
{
    const size_t smem = 3 * (size_t)a.max_M * sizeof(float) + (256 + 8 + 2) * sizeof(unsigned);
    return launch_persistent(compress_nd_kernel, smem, a.n_chunks, sm_count, stream, &a);
}

cudaError_t demo_launch_decode_nd(const DemoNdDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    const size_t smem = 2 * (size_t)a.max_M * sizeof(float) + (((size_t)a.max_M * 2 + 15) & ~(size_t)15);
    return launch_persistent(decode_nd_kernel, smem, a.n_chunks, sm_count, stream, &a);
}
