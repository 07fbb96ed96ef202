// Device-side helpers shared by the fast kernels: mbarrier / TMA wrappers with bounded waits, the
// tensor-table cursor, small warp primitives.
#pragma once

#include <cuda_bf16.h>

#include "demo_internal.h"

namespace fastk {

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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, unsigned parity, long long limit = WAIT_LIMIT_CYCLES)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
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

// 2-D tiled TMA load of one box (coordinates in elements: x along the row, y the row index).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *tmap, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(tmap), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// Pull one box into L2 ahead of its use.
__device__ __forceinline__ void tma_prefetch_2d(const void *tmap, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(tmap), "r"(x), "r"(y) : "memory");
}
// 2-D tiled TMA store of one box from shared memory (bulk-group completion).
__device__ __forceinline__ void tma_store_2d(const void *tmap, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(tmap), "r"(x), "r"(y),
                 "r"(src)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits (the issuing thread's own bulk groups; completes by itself): source read out / fully done.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// The tensor maps live in global memory and are rewritten by the host (a stream-ordered copy) when the
// caller's buffers change: the thread that is about to use one acquires it for the tensor-map proxy first.
__device__ __forceinline__ void tmap_acquire(const void *tmap)
{
    asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(tmap) : "memory");
}
constexpr int TMAP_BYTES = 128;  // sizeof(CUtensorMap)

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
// max of three (one instruction on sm_100)
__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max3abs(float a, float b, float c) { return max3f(fabsf(a), fabsf(b), fabsf(c)); }
__device__ __forceinline__ unsigned mag_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Walks the tensor table as the CTA's chunk ids grow.  The first chunk of the next tensor is kept in a
// register, so that a chunk inside the current tensor costs one comparison and no memory access.
struct EntryCursor {
    int e = 0;
    DemoTensorEntry te;
    long long next_begin = 0;  // chunk_begin of entry e + 1 (or "never")
    bool loaded = false;
    __device__ __forceinline__ void load(const DemoTensorEntry *entries, int n)
    {
        te = entries[e];
        next_begin = (e + 1 < n) ? entries[e + 1].chunk_begin : 0x7fffffffffffffffLL;
    }
    __device__ __forceinline__ void seek(const DemoTensorEntry *entries, int n, long long c)
    {
        if (!loaded) {
            e = demo_find_entry(entries, n, c);
            load(entries, n);
            loaded = true;
            return;
        }
        if (c < next_begin) return;
        while (e + 1 < n && entries[e + 1].chunk_begin <= c) ++e;
        load(entries, n);
    }
};

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

// A CTA hosts NCH independent "slots" of S threads, one chunk each.  Threads of a slot meet at the
// slot's own named barrier (a warp-level barrier when the slot is a single warp); all slots meet once
// per chunk at the CTA barrier, which keeps the warps of the CTA in the same region of the (large,
// fully unrolled) code so that instruction fetches are shared instead of streamed once per warp.
template <int S>
struct SlotBarrier {
    int id;  // named barrier 1..15
    __device__ __forceinline__ void sync() const
    {
        if (S == 32)
            __syncwarp();
        else
            asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(S) : "memory");
    }
    __device__ __forceinline__ bool sync_and(bool pred) const
    {
        if (S == 32) return __all_sync(0xffffffffu, pred);
        unsigned r;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %3, 0;\n\t"
            "bar.red.and.pred p, %1, %2, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(r)
            : "r"(id), "n"(S), "r"((unsigned)pred)
            : "memory");
        return r != 0;
    }
};

// ------------------------------------------------------------------------------------------------
// Exact radix select over the S x S coefficient tile stored at X[u*XS + v] (S threads).  Returns the
// magnitude key of the k-th largest and how many coefficients equal to it belong to the top-k.
// ------------------------------------------------------------------------------------------------
template <int S, int XS>
__device__ __forceinline__ void radix_select_tile(const float *X, int k_eff, unsigned *hist, unsigned *s_state,
                                                  unsigned *thr, unsigned *need_eq, int t, SlotBarrier<S> sb)
{
    if (t == 0) {
        s_state[0] = 0u;
        s_state[1] = (unsigned)k_eff;
    }
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
        for (int i = t; i < 256; i += S) hist[i] = 0u;
        sb.sync();
        const unsigned prefix = s_state[0];
#pragma unroll 1
        for (int v = 0; v < S; ++v) {
            const unsigned key = mag_key(X[t * XS + v]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        sb.sync();
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
        sb.sync();
    }
    *thr = s_state[0];
    *need_eq = s_state[1];
}


// 64 / 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st64(uint32_t taddr, const float (&v)[64])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x64.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, "
        "%33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, "
        "%49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64};" ::"r"(taddr),
        "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), "f"(v[9]),
        "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]), "f"(v[18]),
        "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]),
        "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31]), "f"(v[32]), "f"(v[33]), "f"(v[34]), "f"(v[35]), "f"(v[36]),
        "f"(v[37]), "f"(v[38]), "f"(v[39]), "f"(v[40]), "f"(v[41]), "f"(v[42]), "f"(v[43]), "f"(v[44]), "f"(v[45]),
        "f"(v[46]), "f"(v[47]), "f"(v[48]), "f"(v[49]), "f"(v[50]), "f"(v[51]), "f"(v[52]), "f"(v[53]), "f"(v[54]),
        "f"(v[55]), "f"(v[56]), "f"(v[57]), "f"(v[58]), "f"(v[59]), "f"(v[60]), "f"(v[61]), "f"(v[62]), "f"(v[63])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]),
          "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]),
          "=f"(v[17]), "=f"(v[18]), "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]),
          "=f"(v[25]), "=f"(v[26]), "=f"(v[27]), "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), "f"(v[9]),
        "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]), "f"(v[18]),
        "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]),
        "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
        : "memory");
}
// Tensor memory used as per-thread storage (no MMA): `cols` columns (a power of two >= 32) for the CTA, allocated by
// its first warp; the base address lands in *slot (shared memory).  All threads of the CTA call both functions.
__device__ __forceinline__ uint32_t tmem_alloc_cta(uint32_t *slot, uint32_t cols)
{
    if ((threadIdx.x >> 5) == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return *slot;
}
__device__ __forceinline__ void tmem_free_cta(uint32_t base, uint32_t cols)
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if ((threadIdx.x >> 5) == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}

// ------------------------------------------------------------------------------------------------
// One warp picks the k_eff largest of n_all candidate keys (all >= the bound `lmin`, n_all <= 32 * NK; list order
// is index order).  NK keys per lane, in list order.  Bit by bit, from the first bit where the bound and the
// largest key differ, it looks for a threshold with exactly k_eff keys at or above it and stops as soon as one is
// found; if the bits run out, equal keys straddle the k_eff-th place: keys above the threshold are kept, keys equal
// to it in list order until k_eff are reached.  emit(pos, i) is called for every kept candidate: i its list
// position, pos its place among the kept ones (ascending list order).
// ------------------------------------------------------------------------------------------------
template <int NK, class Where, class Emit>
__device__ __forceinline__ void warp_ballot_select(const unsigned *cand_key, unsigned n_all, unsigned lmin, int k_eff,
                                                   int lane, Where where, Emit emit)
{
    // where(i): storage position of list entry i (the list may sit in several pieces)
    unsigned keys[NK];
    unsigned hi = 0u;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        const unsigned i = (unsigned)j * 32u + lane;
        keys[j] = (i < n_all) ? cand_key[where(i)] : 0u;
        hi = max(hi, keys[j]);
    }
    hi = __reduce_max_sync(0xffffffffu, hi);
    const int wb0 = 31 - __clz((lmin ^ hi) | 1u);
    unsigned thr = lmin & ~((2u << wb0) - 1u);
    unsigned n_ge = n_all;  // every candidate is >= the bound >= thr
#pragma unroll 1
    for (int b = wb0; b >= 0 && n_ge != (unsigned)k_eff; --b) {
        const unsigned cand = thr | (1u << b);
        unsigned cnt = 0;
#pragma unroll
        for (int j = 0; j < NK; ++j) cnt += __popc(__ballot_sync(0xffffffffu, keys[j] >= cand));
        if (cnt >= (unsigned)k_eff) {
            thr = cand;
            n_ge = cnt;
        }
    }
    unsigned gtb[NK], eqb[NK];
    unsigned n_gt = 0;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        gtb[j] = __ballot_sync(0xffffffffu, keys[j] > thr);
        eqb[j] = __ballot_sync(0xffffffffu, keys[j] == thr);
        n_gt += __popc(gtb[j]);
    }
    const unsigned need_eq = (unsigned)k_eff - n_gt;
    const unsigned lt = (1u << lane) - 1u;
    unsigned gt_before = 0, eq_before = 0;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        const unsigned e = eq_before + __popc(eqb[j] & lt);
        if ((keys[j] > thr) || (keys[j] == thr && e < need_eq))
            emit(gt_before + __popc(gtb[j] & lt) + min(e, need_eq), (unsigned)j * 32u + lane);
        gt_before += __popc(gtb[j]);
        eq_before += __popc(eqb[j]);
    }
}

}  // namespace fastk
