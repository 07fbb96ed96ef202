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
// offset = sum_a k_a s_a stride_a (blocking operator).  A tensor has fewer than 2^31 chunks.
__device__ __forceinline__ size_t chunk_base(const DemoNdEntry &e, unsigned lc)
{
    size_t base = 0;
#pragma unroll
    for (int a = DEMO_ND_DIMS - 1; a >= 0; --a) {
        const unsigned q = lc / (unsigned)e.c[a];
        const unsigned k = lc - q * (unsigned)e.c[a];
        lc = q;
        base += (size_t)k * (size_t)e.s[a] * (size_t)e.stride[a];
    }
    return base;
}

// The entry and the base offset of the CTA's current chunk, looked up by one thread (the table is read
// again only when the chunk belongs to another tensor than the previous one).
struct ChunkSlot {
    DemoNdEntry e;
    size_t base;
};

__device__ __forceinline__ void locate_chunk(ChunkSlot *slot, const DemoNdEntry *entries, int n_entries, long long c)
{
    if (threadIdx.x == 0) {
        if (c < slot->e.chunk_begin || c >= slot->e.chunk_end) slot->e = entries[find_nd_entry(entries, n_entries, c)];
        slot->base = chunk_base(slot->e, (unsigned)(c - slot->e.chunk_begin));
    }
    __syncthreads();
}

// Offset of element i (row-major inside the chunk) relative to the chunk's first element.  The
// divisions by the chunk extents are multiplications by inv[a] = ceil(2^32 / s_a), exact for
// i < 2^14 and s_a <= 2^7.
__device__ __forceinline__ size_t elem_offset(const DemoNdEntry &e, int i)
{
    size_t off = 0;
    unsigned r = (unsigned)i;
#pragma unroll
    for (int a = DEMO_ND_DIMS - 1; a >= 0; --a) {
        if (e.s[a] > 1) {
            const unsigned q = __umulhi(r, e.inv[a]);
            off += (size_t)(r - q * (unsigned)e.s[a]) * (size_t)e.stride[a];
            r = q;
        }
    }
    return off;
}

// One axis of the multilinear product on a chunk in shared memory viewed as [outer][s][inner]:
//   dst[o][j][i] = sum_n T[n][j] src[o][n][i]
// with T = C^T for the forward transform (T[n][j] = C[j][n]) and T = C for the inverse; either way the
// threads of a warp that differ in j read neighbouring table entries.  Each thread owns a TU x TV tile
// of outputs: TU along j, TV along i (VI, vector loads) or along o.
template <int TU, int TV, bool VI>
__device__ __forceinline__ void axis_pass(float *__restrict__ dst, const float *__restrict__ src,
                                          const float *__restrict__ T, int s, int inner, int outer)
{
    const int gj = s / TU;
    const int gi = VI ? inner / TV : inner;
    const int go = VI ? outer : outer / TV;
    const int vstep = VI ? 1 : s * inner;  // distance between the TV inputs (and outputs) of a tile
    const int items = go * gj * gi;
    for (int it = threadIdx.x; it < items; it += GEN_THREADS) {
        const int ii = it % gi;
        const int t = it / gi;
        const int j0 = (t % gj) * TU;
        const int oo = t / gj;
        const int o0 = VI ? oo : oo * TV;
        const int i0 = VI ? ii * TV : ii;
        const float *sp = src + (size_t)o0 * s * inner + i0;
        const float *tp = T + j0;
        float acc[TU][TV];
#pragma unroll
        for (int q = 0; q < TU; ++q)
#pragma unroll
            for (int v = 0; v < TV; ++v) acc[q][v] = 0.f;
#pragma unroll 2
        for (int n = 0; n < s; ++n) {
            float tv[TU], sv[TV];
            if constexpr (TU == 4) {  // s, j0 and the table offset are multiples of 4
                const float4 t4 = __ldg(reinterpret_cast<const float4 *>(tp + n * s));
                tv[0] = t4.x, tv[1] = t4.y, tv[2] = t4.z, tv[3] = t4.w;
            } else {
#pragma unroll
                for (int q = 0; q < TU; ++q) tv[q] = __ldg(tp + n * s + q);
            }
            if constexpr (VI && TV == 4) {  // inner and i0 are multiples of 4, the buffers 16-byte aligned
                const float4 s4 = *reinterpret_cast<const float4 *>(sp + n * inner);
                sv[0] = s4.x, sv[1] = s4.y, sv[2] = s4.z, sv[3] = s4.w;
            } else {
#pragma unroll
                for (int v = 0; v < TV; ++v) sv[v] = sp[n * inner + v * vstep];
            }
#pragma unroll
            for (int q = 0; q < TU; ++q)
#pragma unroll
                for (int v = 0; v < TV; ++v) acc[q][v] = fmaf(tv[q], sv[v], acc[q][v]);
        }
        float *dp = dst + (size_t)o0 * s * inner + (size_t)j0 * inner + i0;
#pragma unroll
        for (int q = 0; q < TU; ++q) {
            if constexpr (VI && TV == 4) {
                *reinterpret_cast<float4 *>(dp + q * inner) = make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]);
            } else {
#pragma unroll
                for (int v = 0; v < TV; ++v) dp[q * inner + v * vstep] = acc[q][v];
            }
        }
    }
}

// The last axis with an extent that is a multiple of 4 (inner == 1: the contracted index is contiguous):
// each thread owns 4 outputs along j for 4 consecutive o and reads its inputs four n at a time with
// 16-byte loads -- 8 loads per 64 FMAs.
__device__ __forceinline__ void axis_pass_last(float *__restrict__ dst, const float *__restrict__ src,
                                               const float *__restrict__ T, int s, int outer)
{
    const int gj = s / 4;
    const int items = (outer / 4) * gj;
    for (int it = threadIdx.x; it < items; it += GEN_THREADS) {
        const int j0 = (it % gj) * 4;
        const int o0 = (it / gj) * 4;
        const float *sp = src + (size_t)o0 * s;
        const float *tp = T + j0;
        float acc[4][4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[q][v] = 0.f;
        for (int n = 0; n < s; n += 4) {
            float sv[4][4];  // [v][dn]
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const float4 s4 = *reinterpret_cast<const float4 *>(sp + v * s + n);
                sv[v][0] = s4.x, sv[v][1] = s4.y, sv[v][2] = s4.z, sv[v][3] = s4.w;
            }
#pragma unroll
            for (int dn = 0; dn < 4; ++dn) {
                const float4 t4 = __ldg(reinterpret_cast<const float4 *>(tp + (n + dn) * s));
                const float tv[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int v = 0; v < 4; ++v) acc[q][v] = fmaf(tv[q], sv[v][dn], acc[q][v]);
            }
        }
#pragma unroll
        for (int v = 0; v < 4; ++v)
            *reinterpret_cast<float4 *>(dst + (size_t)(o0 + v) * s + j0) = make_float4(acc[0][v], acc[1][v], acc[2][v], acc[3][v]);
    }
}

template <int TU>
__device__ __forceinline__ void axis_dispatch(float *dst, const float *src, const float *T, int s, int inner, int M)
{
    const int outer = M / (s * inner);
    // 4-wide tiles along i (or o) where the chunk has enough outputs to keep the CTA busy with them
    if (TU == 4 && inner == 1 && M >= 16 * GEN_THREADS / 2 && (outer & 3) == 0)
        axis_pass_last(dst, src, T, s, outer);
    else if (M >= 16 * GEN_THREADS / 2 && (inner & 3) == 0)
        axis_pass<TU, 4, true>(dst, src, T, s, inner, outer);
    else if (M >= 16 * GEN_THREADS / 2 && (outer & 3) == 0)
        axis_pass<TU, 4, false>(dst, src, T, s, inner, outer);
    else
        axis_pass<TU, 1, true>(dst, src, T, s, inner, outer);
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
        const float *T = tables + e.basis[ax] + (inverse ? 0 : s * s);  // [C | C^T] per extent
        if ((s & 3) == 0)
            axis_dispatch<4>(dst, cur, T, s, inner, e.M);
        else
            axis_dispatch<1>(dst, cur, T, s, inner, e.M);
        __syncthreads();
        cur = dst;
    }
    return cur;
}

__global__ void __launch_bounds__(GEN_THREADS) compress_nd_kernel(DemoNdCompressArgs a)
{
    extern __shared__ __align__(16) float smem[];
    float *Bt = smem;
    float *X1 = Bt + a.max_M;
    float *X2 = X1 + a.max_M;
    unsigned *hist = reinterpret_cast<unsigned *>(X2 + a.max_M);  // [256]
    unsigned *warp_tot = hist + 256;                              // [8]
    unsigned *s_state = warp_tot + 8;                             // [2]
    __shared__ ChunkSlot slot;
    const int tid = threadIdx.x;
    if (tid == 0) slot.e.chunk_begin = 1, slot.e.chunk_end = 0;  // no tensor yet

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        locate_chunk(&slot, a.entries, a.n_entries, c);
        const DemoNdEntry &e = slot.e;
        const long long lc = c - e.chunk_begin;
        const size_t base = slot.base;
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
    extern __shared__ __align__(16) float smem[];
    float *St = smem;
    float *X1 = St + a.max_M;
    unsigned short *Cn = reinterpret_cast<unsigned short *>(X1 + a.max_M);  // senders per coordinate (agg == 2)
    __shared__ ChunkSlot slot;
    const int tid = threadIdx.x;
    const bool counts = a.agg == 2;
    if (tid == 0) slot.e.chunk_begin = 1, slot.e.chunk_end = 0;  // no tensor yet

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        locate_chunk(&slot, a.entries, a.n_entries, c);
        const DemoNdEntry &e = slot.e;
        const long long lc = c - e.chunk_begin;
        const size_t base = slot.base;
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
            if (a.sign_ptrs) {  // parameter-server form: hand out sign(R), the workers apply it
                a.sign_ptrs[e.tensor][off] = (signed char)((rv > 0.f) - (rv < 0.f));
                continue;
            }
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
