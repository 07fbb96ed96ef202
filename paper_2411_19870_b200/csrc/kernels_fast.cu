// Fast kernels for 2-D tensors, chunk size S in {32, 64}: S threads own one S x S chunk.
//
// compress (Algorithm 1 worker side / CompressChunks, fused per chunk):
//   bulk-async copies (TMA engine, mbarrier completion) stage the m tile and the g tile in shared
//   memory; thread j forms column j of B = beta*m + g in registers, keeps B in shared memory for
//   the residual, and runs a register-resident fast DCT-II down the column; a shared-memory
//   transpose hands thread u row u for the second pass, after which thread u holds the
//   coefficients Q[u][0..S) in registers.  Exact top-k: the k-th largest of the S per-thread maxima
//   is a lower bound L of the k-th largest coefficient, so only coefficients >= L (a few dozen)
//   are candidates; they are ranked exactly (ties to the lowest index) and written as records in
//   ascending index order.  When the bound is too weak (more than CAP candidates: tied or
//   degenerate chunks) or k > S, an exact radix select over the whole chunk takes over.  The
//   residual uses the sparsity of the kept set: the row stage of the inverse is k rank-1 updates
//   from a cosine table, the column stage one fast DCT-III per thread, then m <- B - IDCT(kept).
// decode (Decompress&Aggregate + update): scatter-add the W payloads in worker order into a shared
//   tile, two fast DCT-III passes, sign, x <- x - lr (sign + wd x).
//
// Every wait on an mbarrier is bounded: on expiry the CTA records DEMO_DEV_TIMEOUT and returns.
#include <cuda_bf16.h>

#include "demo_internal.h"
#include "fast_dct.cuh"

namespace {

constexpr int CAP = 128;                          // candidate capacity of the fast top-k
constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;  // ~1 s

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within WAIT_LIMIT_CYCLES.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, unsigned parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) return false;
    }
    return true;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 1-D bulk async copy global -> shared (16-byte aligned addresses, size a multiple of 16).
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, unsigned bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ unsigned mag_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

template <int S>
struct Cfg {
    static constexpr int XS = S + 4;  // row stride of the transpose tile: conflict-free scalar
                                      // column access and 128-bit row access
    static constexpr int NW = S / 32;
    static constexpr int LOG2S = (S == 64) ? 6 : 5;
};

// Walks the tensor table as the CTA's chunk ids grow.
struct EntryCursor {
    int e = 0;
    DemoTensorEntry te;
    bool loaded = false;
    __device__ __forceinline__ void seek(const DemoTensorEntry *entries, int n, long long c)
    {
        if (!loaded) {
            e = demo_find_entry(entries, n, c);
            te = entries[e];
            loaded = true;
            return;
        }
        bool moved = false;
        while (e + 1 < n && entries[e + 1].chunk_begin <= c) {
            ++e;
            moved = true;
        }
        if (moved) te = entries[e];
    }
};

// ------------------------------------------------------------------------------------------------
// Exact radix select over the S x S coefficient tile stored at X[u*XS + v] (S threads).  Returns the
// magnitude key of the k-th largest and how many coefficients equal to it belong to the top-k.
// ------------------------------------------------------------------------------------------------
template <int S>
__device__ __forceinline__ void radix_select_tile(const float *X, int k_eff, unsigned *hist, unsigned *s_state,
                                                  unsigned *thr, unsigned *need_eq)
{
    constexpr int XS = Cfg<S>::XS;
    const int t = threadIdx.x;
    if (t == 0) {
        s_state[0] = 0u;
        s_state[1] = (unsigned)k_eff;
    }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
        for (int i = t; i < 256; i += S) hist[i] = 0u;
        __syncthreads();
        const unsigned prefix = s_state[0];
        for (int v = 0; v < S; ++v) {
            const unsigned key = mag_key(X[t * XS + v]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (t < 32) {
            const unsigned rem = s_state[1];
            unsigned local = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) local += hist[255 - 8 * t - j];
            unsigned inc = local;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                unsigned n = __shfl_up_sync(0xffffffffu, inc, d);
                if (t >= d) inc += n;
            }
            const unsigned before = inc - local;
            if (before < rem && rem <= inc) {
                unsigned cum = before;
                int b = 255 - 8 * t;
                for (int j = 0; j < 8; ++j, --b) {
                    const unsigned h = hist[b];
                    if (cum + h >= rem) break;
                    cum += h;
                }
                s_state[1] = rem - cum;
                s_state[0] = prefix | ((unsigned)b << shift);
            }
        }
        __syncthreads();
    }
    *thr = s_state[0];
    *need_eq = s_state[1];
}

// Inclusive warp scan.
__device__ __forceinline__ unsigned warp_inclusive_scan(unsigned v, int lane)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned n = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += n;
    }
    return v;
}

template <int S, typename GT>
__global__ void __launch_bounds__(S) compress_fast_kernel(DemoCompressArgs a)
{
    using C = Cfg<S>;
    constexpr int XS = C::XS, NW = C::NW, LOG2S = C::LOG2S;
    constexpr unsigned TILE_BYTES = S * S * sizeof(float) + S * S * sizeof(GT);

    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *Bt = reinterpret_cast<float *>(smem_raw);             // [S*S]   m tile, then B
    float *X = Bt + S * S;                                       // [S*XS]  g staging / transpose / Q / T
    float *costab = X + S * XS;                                  // [4*S]   cos(pi t / (2S))
    float *tmax = costab + 4 * S;                                // [S]
    int *cand_idx = reinterpret_cast<int *>(tmax + S);           // [CAP]
    float *cand_val = reinterpret_cast<float *>(cand_idx + CAP); // [CAP]
    unsigned *hist = reinterpret_cast<unsigned *>(cand_idx);     // [256] aliases the candidate arrays
    DemoRecord *recs = reinterpret_cast<DemoRecord *>(cand_val + CAP);  // [64]
    unsigned *misc = reinterpret_cast<unsigned *>(recs + 64);    // [16]
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(misc + 16);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const uint32_t bar = smem_u32(bar_mem);

    for (int i = t; i < 4 * S; i += S) costab[i] = cospif((float)i / (float)(2 * S));
    if (t == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();  // make the initialised barrier visible to the async proxy
    }
    __syncthreads();
    fence_proxy_async();

    EntryCursor cur;
    float *m_ptr = nullptr;
    const GT *g_ptr = nullptr;
    int cached_tensor = -1;
    unsigned phase = 0;

    auto issue_loads = [&](long long c) {
        cur.seek(a.entries, a.n_entries, c);
        if (cur.te.tensor != cached_tensor) {
            cached_tensor = cur.te.tensor;
            m_ptr = a.m_ptrs[cached_tensor];
            g_ptr = reinterpret_cast<const GT *>(a.g_ptrs[cached_tensor]);
        }
        const long long lc = c - cur.te.chunk_begin;
        const long long k0 = lc / cur.te.c1;
        const int k1 = (int)(lc - k0 * cur.te.c1);
        const size_t off = ((size_t)k0 * S + t) * (size_t)cur.te.n1 + (size_t)k1 * S;  // row t of the tile
        if (t == 0) mbar_expect_tx(bar, TILE_BYTES);
        fence_proxy_async();
        bulk_g2s(smem_u32(Bt + t * S), m_ptr + off, S * sizeof(float), bar);
        bulk_g2s(smem_u32(reinterpret_cast<GT *>(X) + t * S), g_ptr + off, S * sizeof(GT), bar);
    };

    long long c = blockIdx.x;
    if (c < a.n_chunks) issue_loads(c);

    for (; c < a.n_chunks; c += gridDim.x) {
        // the cursor points at chunk c (issue_loads(c) ran last)
        const DemoTensorEntry te = cur.te;
        const long long lc = c - te.chunk_begin;
        const long long k0 = lc / te.c1;
        const int k1 = (int)(lc - k0 * te.c1);
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ m = m_ptr;
        const int k_eff = te.k_eff;
        DemoRecord *rec = a.payload + te.rec_begin + lc * (long long)k_eff;

        const bool arrived = mbar_wait_bounded(bar, phase);
        phase ^= 1u;
        if (!__syncthreads_and(arrived)) {
            if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);  // give copies in flight one more bounded chance to land
            return;
        }

        // ---- momentum update on column t, first DCT pass down the column -------------------------
        {
            float x[S];
            const GT *gs = reinterpret_cast<const GT *>(X);
#pragma unroll
            for (int i = 0; i < S; ++i) x[i] = fmaf(a.beta, Bt[i * S + t], to_f32(gs[i * S + t]));
            __syncthreads();  // every thread has consumed the g staging area inside X
#pragma unroll
            for (int i = 0; i < S; ++i) Bt[i * S + t] = x[i];
            fdct::dct2_ortho<S>(x);
#pragma unroll
            for (int u = 0; u < S; ++u) X[u * XS + t] = x[u];
        }
        __syncthreads();

        // ---- second DCT pass along row t: q[v] = Q[t][v] -----------------------------------------
        float q[S];
        {
            const float4 *row = reinterpret_cast<const float4 *>(X + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) {
                const float4 f = row[v4];
                q[4 * v4 + 0] = f.x;
                q[4 * v4 + 1] = f.y;
                q[4 * v4 + 2] = f.z;
                q[4 * v4 + 3] = f.w;
            }
        }
        fdct::dct2_ortho<S>(q);

        // ---- top-k ------------------------------------------------------------------------------
        bool use_fallback = (k_eff > S);
        unsigned n_c = 0, off = 0;
        unsigned long long mask = 0ull;
        if (!use_fallback) {
            float tm = 0.f;
#pragma unroll
            for (int v = 0; v < S; ++v) tm = fmaxf(tm, fabsf(q[v]));
            // bitonic sort (descending) of the 32 per-thread maxima of this warp
            float sv = tm;
#pragma unroll
            for (int k2 = 2; k2 <= 32; k2 <<= 1) {
#pragma unroll
                for (int j = k2 >> 1; j > 0; j >>= 1) {
                    const float other = __shfl_xor_sync(0xffffffffu, sv, j);
                    const bool keep_max = ((lane & j) == 0) == ((lane & k2) == 0);
                    sv = keep_max ? fmaxf(sv, other) : fminf(sv, other);
                }
            }
            float L;
            if (NW == 1) {
                L = __shfl_sync(0xffffffffu, sv, k_eff - 1);
            } else {
                tmax[t] = sv;
                __syncthreads();
                // rank of this element in the union of the two descending lists (strict order:
                // equal values of warp 0 come first)
                const float *other = tmax + (warp ^ 1) * 32;
                int lo = 0, hi = 32;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    const float o = other[mid];
                    const bool before = (warp == 0) ? (o > sv) : (o >= sv);
                    if (before)
                        lo = mid + 1;
                    else
                        hi = mid;
                }
                if (lane + lo == k_eff - 1) reinterpret_cast<float *>(misc)[8] = sv;
                __syncthreads();
                L = reinterpret_cast<float *>(misc)[8];
            }
            // candidates: coefficients with magnitude >= L (at least k_eff of them exist)
            unsigned mlo = 0u, mhi = 0u;
#pragma unroll
            for (int v = 0; v < S; ++v) {
                const bool p = fabsf(q[v]) >= L;
                if (v < 32)
                    mlo |= p ? (1u << v) : 0u;
                else
                    mhi |= p ? (1u << (v - 32)) : 0u;
            }
            mask = ((unsigned long long)mhi << 32) | mlo;
            const unsigned cnt = __popc(mlo) + __popc(mhi);
            const unsigned inc = warp_inclusive_scan(cnt, lane);
            if (lane == 31) misc[warp] = inc;
            __syncthreads();
            off = inc - cnt;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                if (w < warp) off += misc[w];
                n_c += misc[w];
            }
            use_fallback = (n_c > CAP);
        }
        // stash the coefficients of row t (own row: no hazard with other threads)
        {
            float4 *row = reinterpret_cast<float4 *>(X + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(q[4 * v4], q[4 * v4 + 1], q[4 * v4 + 2], q[4 * v4 + 3]);
        }

        if (!use_fallback) {
            unsigned o = off;
            while (mask) {
                const int v = __ffsll((long long)mask) - 1;
                mask &= mask - 1ull;
                cand_idx[o] = t * S + v;
                cand_val[o] = X[t * XS + v];
                ++o;
            }
            __syncthreads();
            // exact rank among the candidates: larger magnitude first, then lower index (the list
            // is in ascending index order, so the list position stands for the index)
            constexpr int ITER = CAP / S;
            bool sel[ITER];
            unsigned pre[ITER];
#pragma unroll
            for (int it = 0; it < ITER; ++it) {
                const unsigned ci = it * S + t;
                sel[it] = false;
                if (ci < n_c) {
                    const unsigned key = mag_key(cand_val[ci]);
                    unsigned rank = 0;
                    for (unsigned c2 = 0; c2 < n_c; ++c2) {
                        const unsigned k2 = mag_key(cand_val[c2]);
                        rank += (k2 > key) || (k2 == key && c2 < ci);
                    }
                    sel[it] = rank < (unsigned)k_eff;
                }
                const unsigned bal = __ballot_sync(0xffffffffu, sel[it]);
                pre[it] = __popc(bal & ((1u << lane) - 1u));
                if (lane == 0) misc[4 + it * NW + warp] = __popc(bal);
            }
            __syncthreads();
#pragma unroll
            for (int it = 0; it < ITER; ++it) {
                if (sel[it]) {
                    unsigned pos = pre[it];
                    for (int g = 0; g < it * NW + warp; ++g) pos += misc[4 + g];
                    DemoRecord r;
                    r.idx = cand_idx[it * S + t];
                    r.val = cand_val[it * S + t];
                    rec[pos] = r;
                    recs[pos] = r;  // k_eff <= S <= 64 on this path
                }
            }
        } else {
            __syncthreads();  // coefficient tile complete in X
            unsigned thr, need_eq;
            radix_select_tile<S>(X, k_eff, hist, misc, &thr, &need_eq);
            unsigned gt = 0, eq = 0;
            for (int v = 0; v < S; ++v) {
                const unsigned key = mag_key(X[t * XS + v]);
                gt += key > thr;
                eq += key == thr;
            }
            const unsigned packed = gt | (eq << 16);
            const unsigned inc = warp_inclusive_scan(packed, lane);
            __syncthreads();  // radix_select_tile's last reads of misc are done
            if (lane == 31) misc[warp] = inc;
            __syncthreads();
            unsigned before = inc - packed;
#pragma unroll
            for (int w = 0; w < NW; ++w)
                if (w < warp) before += misc[w];
            unsigned gb = before & 0xffffu, eb = before >> 16;
            for (int v = 0; v < S; ++v) {
                const float val = X[t * XS + v];
                const unsigned key = mag_key(val);
                bool s = false;
                unsigned pos = 0;
                if (key > thr) {
                    pos = gb + min(eb, need_eq);
                    ++gb;
                    s = true;
                } else if (key == thr) {
                    if (eb < need_eq) {
                        pos = gb + eb;
                        s = true;
                    }
                    ++eb;
                }
                if (s) {
                    DemoRecord r;
                    r.idx = t * S + v;
                    r.val = val;
                    rec[pos] = r;
                    if (k_eff <= 64) recs[pos] = r;
                }
            }
        }
        __syncthreads();  // records complete (shared list and global payload); X is free

        // ---- residual: row stage of the inverse from the k_eff records, sparse ------------------
        {
            float4 *row = reinterpret_cast<float4 *>(X + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        __syncthreads();
        {
            constexpr float sc = (float)fdct::ScaleOrtho<S>::value, dc = fdct::dc_scale<S>();
            const int tw = 2 * t + 1;
            float acc = 0.f;
            int cur_u = -1;
            for (int r = 0; r < k_eff; ++r) {
                const DemoRecord rc = (k_eff <= 64) ? recs[r] : rec[r];
                const int u = rc.idx >> LOG2S, v = rc.idx & (S - 1);
                if (u != cur_u) {
                    if (cur_u >= 0) X[cur_u * XS + t] = acc;
                    acc = 0.f;
                    cur_u = u;
                }
                const float sv = rc.val * (v == 0 ? dc : sc);
                acc = fmaf(sv, costab[(tw * v) & (4 * S - 1)], acc);  // T[u][t] += val * C[v][t]
            }
            if (cur_u >= 0) X[cur_u * XS + t] = acc;
        }
        // column t of T was written by this thread only: no barrier needed before reading it back
        {
            float r[S];
#pragma unroll
            for (int u = 0; u < S; ++u) r[u] = X[u * XS + t];
            fdct::dct3_ortho<S>(r);
#pragma unroll
            for (int i = 0; i < S; ++i) m[base + (size_t)i * te.n1 + t] = Bt[i * S + t] - r[i];
        }
        __syncthreads();  // Bt and X are free again
        const long long nc = c + gridDim.x;
        if (nc < a.n_chunks) issue_loads(nc);
    }
}

template <int S>
__global__ void __launch_bounds__(S) decode_fast_kernel(DemoDecodeArgs a)
{
    using C = Cfg<S>;
    constexpr int XS = C::XS;
    constexpr int M = S * S;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *Xt = reinterpret_cast<float *>(smem_raw);  // [S*S]  x tile
    float *St = Xt + S * S;                           // [S*XS] aggregate, then row-stage output
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(St + S * XS);

    const int t = threadIdx.x;
    const uint32_t bar = smem_u32(bar_mem);
    if (t == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();  // make the initialised barrier visible to the async proxy
    }
    __syncthreads();
    fence_proxy_async();

    EntryCursor cur;
    float *x_ptr = nullptr;
    int cached_tensor = -1;
    unsigned phase = 0;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        cur.seek(a.entries, a.n_entries, c);
        const DemoTensorEntry te = cur.te;
        if (te.tensor != cached_tensor) {
            cached_tensor = te.tensor;
            x_ptr = a.x_ptrs[cached_tensor];
        }
        const long long lc = c - te.chunk_begin;
        const long long k0 = lc / te.c1;
        const int k1 = (int)(lc - k0 * te.c1);
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ x = x_ptr;
        const int k_eff = te.k_eff;
        const long long rec_off = te.rec_begin + lc * (long long)k_eff;

        // stage the x tile while the aggregate is built
        if (t == 0) mbar_expect_tx(bar, S * S * sizeof(float));
        fence_proxy_async();
        bulk_g2s(smem_u32(Xt + t * S), x + base + (size_t)t * te.n1, S * sizeof(float), bar);

        {
            float4 *row = reinterpret_cast<float4 *>(St + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        __syncthreads();
        // S = sum over workers in worker order; a barrier per worker fixes the order of additions
        for (int w = 0; w < a.W; ++w) {
            const DemoRecord *rec = a.payloads[w] + rec_off;
            for (int i = t; i < k_eff; i += S) {
                const DemoRecord r = rec[i];
                if ((unsigned)r.idx < (unsigned)M)
                    St[(r.idx >> C::LOG2S) * XS + (r.idx & (S - 1))] += r.val;
                else
                    atomicMax(a.status, DEMO_DEV_PAYLOAD);
            }
            __syncthreads();
        }
        // inverse along the row (thread t owns row t, in place)
        {
            float r[S];
            float4 *row = reinterpret_cast<float4 *>(St + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) {
                const float4 f = row[v4];
                r[4 * v4 + 0] = f.x;
                r[4 * v4 + 1] = f.y;
                r[4 * v4 + 2] = f.z;
                r[4 * v4 + 3] = f.w;
            }
            fdct::dct3_ortho<S>(r);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(r[4 * v4], r[4 * v4 + 1], r[4 * v4 + 2], r[4 * v4 + 3]);
        }
        __syncthreads();
        const bool arrived = mbar_wait_bounded(bar, phase);
        phase ^= 1u;
        if (!__syncthreads_and(arrived)) {
            if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);
            return;
        }
        // inverse down column t, sign, update
        {
            float r[S];
#pragma unroll
            for (int u = 0; u < S; ++u) r[u] = St[u * XS + t];
            fdct::dct3_ortho<S>(r);
#pragma unroll
            for (int i = 0; i < S; ++i) {
                const float rv = r[i];
                const float sg = (float)((rv > 0.f) - (rv < 0.f));
                const float xv = Xt[i * S + t];
                x[base + (size_t)i * te.n1 + t] = fmaf(-a.lr, fmaf(a.wd, xv, sg), xv);
            }
        }
        __syncthreads();  // Xt and St are free again
    }
}

template <int S>
constexpr size_t compress_smem()
{
    return (size_t)S * S * 4 + (size_t)S * Cfg<S>::XS * 4 + 4 * S * 4 + S * 4 + CAP * 8 + 64 * 8 + 16 * 4 + 16;
}
template <int S>
constexpr size_t decode_smem()
{
    return (size_t)S * S * 4 + (size_t)S * Cfg<S>::XS * 4 + 16;
}

template <typename K>
cudaError_t launch(K kernel, int threads, size_t smem, long long n_chunks, int sm_count, cudaStream_t stream,
                   const void *args)
{
    if (n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    int per_sm = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count * per_sm;
    if (grid > n_chunks) grid = n_chunks;
    void *params[] = {const_cast<void *>(args)};
    return cudaLaunchKernel((const void *)kernel, dim3((unsigned)grid), dim3(threads), params, smem, stream);
}

}  // namespace

bool demo_fast_supported(int s) { return s == 64 || s == 32; }

cudaError_t demo_launch_compress_fast(int s, const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    if (s == 64) {
        if (a.grad_bf16)
            return launch(compress_fast_kernel<64, __nv_bfloat16>, 64, compress_smem<64>(), a.n_chunks, sm_count, stream, &a);
        return launch(compress_fast_kernel<64, float>, 64, compress_smem<64>(), a.n_chunks, sm_count, stream, &a);
    }
    if (s == 32) {
        if (a.grad_bf16)
            return launch(compress_fast_kernel<32, __nv_bfloat16>, 32, compress_smem<32>(), a.n_chunks, sm_count, stream, &a);
        return launch(compress_fast_kernel<32, float>, 32, compress_smem<32>(), a.n_chunks, sm_count, stream, &a);
    }
    return cudaErrorInvalidValue;
}

cudaError_t demo_launch_decode_fast(int s, const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    if (s == 64) return launch(decode_fast_kernel<64>, 64, decode_smem<64>(), a.n_chunks, sm_count, stream, &a);
    if (s == 32) return launch(decode_fast_kernel<32>, 32, decode_smem<32>(), a.n_chunks, sm_count, stream, &a);
    return cudaErrorInvalidValue;
}
