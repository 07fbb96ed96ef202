// Tensor-core kernels for caller-supplied orthonormal bases, chunk size 64 (Section 4.2, "Choice of
// Linear Projections": identity, random orthonormal projection).  With an arbitrary basis P the chunk
// transform Q = P B P^T is a dense contraction with no fast factorisation, so it runs on the 5th
// generation tensor cores: tcgen05.mma (kind::tf32) with fp32 accumulators in tensor memory.
//
// A group of 128 threads works on a PAIR of chunks stacked to M = 128; thread (c, r) owns row r of
// chunk c.  A CTA holds two such groups (own operand tiles, mbarrier and tensor-memory columns) that run
// independently, so that one group's global-memory and tensor-core latencies hide behind the other's
// work.  Every stage is  D[128 x 64] = A * basis  with
//   A      the pair's data tile, MN-major: the rows of the tile are the K-rows of the operand, 128 bytes
//          each, in the 128-byte swizzle with 32-byte atoms (the layout MN-major TF32 operands need);
//          each thread writes its own row, so no transpose is ever made;
//   basis  P as the K-major operand (contracts over the columns of P: forward) or as the MN-major
//          operand (contracts over the rows of P: inverse).
// Stage 1 turns rows i into columns of the result (lane (c, j) of tensor memory holds (P B)[.][j]); the
// thread that reads that lane writes it back as K-row j of the next operand; stage 2 leaves thread
// (c, u) with row u of Q.  fp32 accuracy comes from 3xTF32: every operand is split into hi = tf32(v)
// and lo = tf32(v - hi) and the stage accumulates lo*hi + hi*lo + hi*hi (24 MMAs of 128 x 64 x 8).
// Top-k is the exact radix select of the other kernel families; the kept coefficients go back through
// two inverse stages as a (mostly zero) dense tile.  Global memory is read and written tile-wise,
// coalesced, through a plain fp32 tile in shared memory that each thread then reads by row.  Every wait
// is bounded: on expiry the CTA records
// DEMO_DEV_TIMEOUT, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "demo_internal.h"
#include "fast_common.cuh"

namespace {

using namespace fastk;

constexpr int S = 64;
constexpr int M = S * S;
constexpr int PAIR_THREADS = 128;
constexpr int GROUPS = 2;                  // pair groups per CTA
constexpr int TC_THREADS = GROUPS * PAIR_THREADS;
constexpr int BLK = 8192;   // one [64 rows][128 bytes] operand block
constexpr int XS = S + 4;   // row stride of the plain fp32 tiles (coefficients, aggregate, staging)
constexpr int TMEM_COLS_PER_GROUP = 128;
constexpr int TMEM_COLS = GROUPS * TMEM_COLS_PER_GROUP;

// shared memory (offsets from a 1024-byte aligned base)
constexpr int OP_BYTES = 8 * BLK;          // per group: hi tile (4 blocks: (chunk c, column block cb) -> 2c + cb), lo tile
constexpr int OFF_OP_HI = 0;
constexpr int OFF_OP_LO = 4 * BLK;
constexpr int OFF_BK_HI = GROUPS * OP_BYTES;      // basis, K-major operand (2 blocks)
constexpr int OFF_BK_LO = OFF_BK_HI + 2 * BLK;
constexpr int OFF_BM_HI = OFF_BK_LO + 2 * BLK;    // basis, MN-major operand (2 blocks)
constexpr int OFF_BM_LO = OFF_BM_HI + 2 * BLK;
constexpr int OFF_MISC = OFF_BM_LO + 2 * BLK;     // per chunk: hist[256], state[16]; then mbarriers, tensor-memory slot
constexpr int CAPT = 128;                        // candidate capacity of the fast top-k
constexpr int HIST_WORDS = 2 * (CAPT + 4);       // radix histogram [256], or candidate keys [CAPT + 4] + indices [CAPT + 4]
constexpr int MISC_PER_CHUNK = (HIST_WORDS + 80 + 128) * 4;  // + misc[80] + rowmask[128]
constexpr int OFF_BARS = OFF_MISC + 2 * GROUPS * MISC_PER_CHUNK;
constexpr int TC_SMEM_BYTES = OFF_BARS + 64 + 1024;  // + alignment slack

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ float tf32_rn(float v)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return __uint_as_float(r);
}

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4), descriptor
// version 1, layout 2 = 128-byte swizzle, 1 = 128-byte swizzle with 32-byte atoms.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout)
{
    uint64_t d = (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)layout << 61;
    return d;
}
// Instruction descriptor: D fp32, A and B tf32, A MN-major, B K- or MN-major, N = 64, M = 128.
__device__ __forceinline__ constexpr uint32_t instr_desc(int b_mn)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((uint32_t)b_mn << 16) | ((uint32_t)(S >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 64 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float *v)
{
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
        "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
        "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]),
          "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]),
          "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]),
          "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]),
          "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}

// Byte offset of the 16-byte piece q (0..7) of row r in block (2c + cb): MN = true is the 32-byte-atom
// swizzle of MN-major TF32 operands, MN = false the plain 128-byte swizzle of K-major ones.
template <bool MN>
__device__ __forceinline__ uint32_t op_off(int c, int cb, int r, int q)
{
    if (MN) return (2 * c + cb) * BLK + r * 128 + ((((q >> 1) ^ (r & 3)) << 5) | ((q & 1) << 4));
    return (2 * c + cb) * BLK + r * 128 + ((q ^ (r & 7)) << 4);
}
// Row r of chunk c (64 floats) split into the hi and lo operand tiles.
template <bool MN>
__device__ __forceinline__ void write_split_row(unsigned char *hi, unsigned char *lo, int c, int r, const float *v)
{
#pragma unroll
    for (int cb = 0; cb < 2; ++cb)
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float *p = v + cb * 32 + q * 4;
            float4 h, l;
            h.x = tf32_rn(p[0]);
            h.y = tf32_rn(p[1]);
            h.z = tf32_rn(p[2]);
            h.w = tf32_rn(p[3]);
            l.x = tf32_rn(p[0] - h.x);
            l.y = tf32_rn(p[1] - h.y);
            l.z = tf32_rn(p[2] - h.z);
            l.w = tf32_rn(p[3] - h.w);
            *reinterpret_cast<float4 *>(hi + op_off<MN>(c, cb, r, q)) = h;
            *reinterpret_cast<float4 *>(lo + op_off<MN>(c, cb, r, q)) = l;
        }
}

// One stage, issued by one thread: D = (A_hi + A_lo) * (B_hi + B_lo) without the lo * lo term, small
// products first.  K = 64 in eight steps of 8: a step is 8 K-rows (1024 bytes) of an MN-major operand,
// 32 bytes inside a 128-byte row of the K-major basis (second half of K one block further).
__device__ __forceinline__ void issue_stage(uint32_t d_tmem, uint32_t a_hi, uint32_t a_lo, uint32_t b_hi, uint32_t b_lo, int b_mn)
{
    const uint32_t idesc = instr_desc(b_mn);
    uint32_t acc = 0;
#pragma unroll 1
    for (int prod = 0; prod < 3; ++prod) {
        const uint32_t a = (prod == 0) ? a_lo : a_hi;
        const uint32_t b = (prod == 1) ? b_lo : b_hi;
#pragma unroll 1
        for (int kk = 0; kk < 8; ++kk) {
            const uint64_t ad = smem_desc(a + kk * 1024, BLK, 512, 1);
            const uint64_t bd = b_mn ? smem_desc(b + kk * 1024, BLK, 512, 1)
                                     : smem_desc(b + (kk >> 2) * BLK + (kk & 3) * 32, 16, 1024, 2);
            umma_tf32(d_tmem, ad, bd, idesc, acc);
            acc = 1;
        }
    }
}

// Common frame of both kernels: aligned shared memory, per-group mbarrier, tensor memory, split basis tiles.
struct TcFrame {
    unsigned char *sm;   // aligned base
    unsigned char *op;   // this group's operand tiles
    uint32_t bar, tmem_base, lane_addr;
    unsigned phase;
    int g, pt;           // pair group, thread inside the group
};

__device__ __forceinline__ void tc_setup(TcFrame &f, unsigned char *raw, const float *basis, bool need_k_major)
{
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t raw_s = smem_u32(raw);
    f.sm = raw + (((raw_s + 1023u) & ~1023u) - raw_s);
    f.g = tid / PAIR_THREADS;
    f.pt = tid % PAIR_THREADS;
    f.op = f.sm + f.g * OP_BYTES;
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(f.sm + OFF_BARS);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_mem + GROUPS);
    f.bar = smem_u32(bar_mem + f.g);
    f.phase = 0;
    if (f.pt == 0) {
        mbar_init(f.bar, 1);
        fence_proxy_async();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid < S) {
        float v[S];
#pragma unroll
        for (int j4 = 0; j4 < S / 4; ++j4) {
            const float4 p = __ldg(reinterpret_cast<const float4 *>(basis + tid * S) + j4);
            v[4 * j4] = p.x;
            v[4 * j4 + 1] = p.y;
            v[4 * j4 + 2] = p.z;
            v[4 * j4 + 3] = p.w;
        }
        if (need_k_major) write_split_row<false>(f.sm + OFF_BK_HI, f.sm + OFF_BK_LO, 0, tid, v);
        write_split_row<true>(f.sm + OFF_BM_HI, f.sm + OFF_BM_LO, 0, tid, v);
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    f.tmem_base = *tmem_slot + (uint32_t)(f.g * TMEM_COLS_PER_GROUP);
    f.lane_addr = f.tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
}

__device__ __forceinline__ void tc_teardown(const TcFrame &f)
{
    tc_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(f.tmem_base - (uint32_t)(f.g * TMEM_COLS_PER_GROUP)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
}

// Two chained stages on the pair: on entry every thread holds its row in v and the group's operand tiles
// are free; on return it holds row r of (forward, b_mn = 0) P X P^T or (inverse, b_mn = 1) P^T X P, and
// the tiles are free again.  False if a wait expired.
__device__ __forceinline__ bool tc_transform(TcFrame &f, const SlotBarrier<PAIR_THREADS> &pb, int c, int r, float *v, int b_mn)
{
    unsigned char *hi = f.op + OFF_OP_HI, *lo = f.op + OFF_OP_LO;
    const uint32_t b_hi = smem_u32(f.sm + (b_mn ? OFF_BM_HI : OFF_BK_HI));
    const uint32_t b_lo = smem_u32(f.sm + (b_mn ? OFF_BM_LO : OFF_BK_LO));
#pragma unroll 1
    for (int stage = 0; stage < 2; ++stage) {
        write_split_row<true>(hi, lo, c, r, v);
        fence_proxy_async();   // generic-proxy writes -> visible to the tensor core's reads
        tc_fence_before();
        pb.sync();
        if (f.pt == 0) {
            tc_fence_after();
            issue_stage(f.tmem_base + stage * S, smem_u32(hi), smem_u32(lo), b_hi, b_lo, b_mn);
            umma_commit(f.bar);
        }
        const bool done = mbar_wait_bounded(f.bar, f.phase);
        f.phase ^= 1u;
        if (!pb.sync_and(done)) return false;
        tc_fence_after();
        tmem_ld64(f.lane_addr + stage * S, v);
    }
    tc_fence_before();
    return true;
}

struct ChunkRef {
    DemoTensorEntry te;
    long long lc;
    size_t tile_off;  // element offset of the tile's first element inside the tensor
    bool valid;
};
__device__ __forceinline__ ChunkRef locate(const DemoTensorEntry *entries, int n_entries, long long n_chunks, long long chunk)
{
    ChunkRef cr;
    cr.valid = chunk < n_chunks;
    cr.lc = 0;
    cr.tile_off = 0;
    if (cr.valid) {
        cr.te = entries[demo_find_entry(entries, n_entries, chunk)];
        cr.lc = chunk - cr.te.chunk_begin;
        const long long k0 = cr.lc / cr.te.c1;
        const int k1 = (int)(cr.lc - k0 * cr.te.c1);
        cr.tile_off = (size_t)k0 * S * (size_t)cr.te.n1 + (size_t)k1 * S;
    } else {
        cr.te = entries[0];
    }
    return cr;
}

// The 64 threads of a chunk move its tile between global memory and the plain fp32 tile T[row * XS + col]
// in 16 sweeps: in sweep `it` thread t handles the 16 bytes at row 4 it + t / 16, columns 4 (t % 16) ..,
// so that 16 threads cover one 256-byte row of the tile.
__device__ __forceinline__ int sweep_row(int it, int t) { return 4 * it + (t >> 4); }
__device__ __forceinline__ int sweep_col(int t) { return 4 * (t & 15); }

__device__ __forceinline__ void read_own_row(const float *T, int r, float *v)
{
#pragma unroll
    for (int j4 = 0; j4 < S / 4; ++j4) {
        const float4 w = reinterpret_cast<const float4 *>(T + r * XS)[j4];
        v[4 * j4] = w.x;
        v[4 * j4 + 1] = w.y;
        v[4 * j4 + 2] = w.z;
        v[4 * j4 + 3] = w.w;
    }
}
__device__ __forceinline__ void write_own_row(float *T, int r, const float *v)
{
#pragma unroll
    for (int j4 = 0; j4 < S / 4; ++j4)
        reinterpret_cast<float4 *>(T + r * XS)[j4] = make_float4(v[4 * j4], v[4 * j4 + 1], v[4 * j4 + 2], v[4 * j4 + 3]);
}

__global__ void __launch_bounds__(TC_THREADS, 1) compress_tc_kernel(DemoCompressArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    TcFrame f;
    tc_setup(f, smem_raw, a.C, true);
    const int c = f.pt >> 6, r = f.pt & 63, lane = f.pt & 31, warp2 = (f.pt >> 5) & 1;
    const SlotBarrier<PAIR_THREADS> pb{1 + f.g};          // the 128 threads of the pair
    const SlotBarrier<S> sb{1 + GROUPS + 2 * f.g + c};    // the 64 threads of one chunk
    float *X = reinterpret_cast<float *>(f.op + (c ? OFF_OP_LO : OFF_OP_HI));  // plain tile of chunk c (aliases the operands)
    unsigned *hist = reinterpret_cast<unsigned *>(f.sm + OFF_MISC + (2 * f.g + c) * MISC_PER_CHUNK);
    unsigned *misc = hist + HIST_WORDS;  // [80]: counts, select state, the 64 row maxima
    unsigned *rowmask = misc + 80;     // [128]: per row, the kept coefficients as a 64-bit mask
    bool ok = true;

    const long long n_pairs = (a.n_chunks + 1) / 2;
    for (long long p = (long long)blockIdx.x * GROUPS + f.g; p < n_pairs; p += (long long)gridDim.x * GROUPS) {
        const ChunkRef cr = locate(a.entries, a.n_entries, a.n_chunks, 2 * p + c);
        const int k_eff = cr.te.k_eff;
        const size_t n1 = (size_t)cr.te.n1;
        float *m_tile = a.m_ptrs[cr.te.tensor] + cr.tile_off;
        {
            // pull the next pair's tiles into L2 while this pair is worked on: 64 threads x 3 lines of 128 bytes
            // cover the 64 x 256 bytes of m and the 64 x 128 (bf16) or 64 x 256 (fp32) bytes of g
            const ChunkRef nx = locate(a.entries, a.n_entries, a.n_chunks, 2 * (p + (long long)gridDim.x * GROUPS) + c);
            if (nx.valid) {
                const char *nm = reinterpret_cast<const char *>(a.m_ptrs[nx.te.tensor] + nx.tile_off) +
                                 (size_t)r * nx.te.n1 * sizeof(float);
                const size_t gsz = a.grad_bf16 ? 2 : 4;
                const char *ng = static_cast<const char *>(a.g_ptrs[nx.te.tensor]) + (nx.tile_off + (size_t)r * nx.te.n1) * gsz;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nm));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nm + 128));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(ng));
                if (!a.grad_bf16) asm volatile("prefetch.global.L2 [%0];" ::"l"(ng + 128));
            }
        }
        float b[S], v[S];
        if (cr.valid) {
            // momentum update, tile-wise and coalesced:  B = beta * m + g  (Algorithm 1, worker side)
            if (a.grad_bf16) {
                const __nv_bfloat16 *g_tile = reinterpret_cast<const __nv_bfloat16 *>(a.g_ptrs[cr.te.tensor]) + cr.tile_off;
#pragma unroll
                for (int it = 0; it < 16; ++it) {
                    const size_t off = (size_t)sweep_row(it, r) * n1 + sweep_col(r);
                    const float4 mv = *reinterpret_cast<const float4 *>(m_tile + off);
                    const uint2 gw = *reinterpret_cast<const uint2 *>(g_tile + off);
                    float4 bv;
                    bv.x = fmaf(a.beta, mv.x, __uint_as_float(gw.x << 16));
                    bv.y = fmaf(a.beta, mv.y, __uint_as_float(gw.x & 0xffff0000u));
                    bv.z = fmaf(a.beta, mv.z, __uint_as_float(gw.y << 16));
                    bv.w = fmaf(a.beta, mv.w, __uint_as_float(gw.y & 0xffff0000u));
                    *reinterpret_cast<float4 *>(X + sweep_row(it, r) * XS + sweep_col(r)) = bv;
                }
            } else {
                const float *g_tile = reinterpret_cast<const float *>(a.g_ptrs[cr.te.tensor]) + cr.tile_off;
#pragma unroll
                for (int it = 0; it < 16; ++it) {
                    const size_t off = (size_t)sweep_row(it, r) * n1 + sweep_col(r);
                    const float4 mv = *reinterpret_cast<const float4 *>(m_tile + off);
                    const float4 gv = *reinterpret_cast<const float4 *>(g_tile + off);
                    *reinterpret_cast<float4 *>(X + sweep_row(it, r) * XS + sweep_col(r)) =
                        make_float4(fmaf(a.beta, mv.x, gv.x), fmaf(a.beta, mv.y, gv.y), fmaf(a.beta, mv.z, gv.z),
                                    fmaf(a.beta, mv.w, gv.w));
                }
            }
            sb.sync();
            read_own_row(X, r, b);
        } else {
#pragma unroll
            for (int j = 0; j < S; ++j) b[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < S; ++j) v[j] = b[j];
        pb.sync();  // every row has been read: the tiles become operand space

        // ---- Q = P B P^T on the tensor cores; thread (c, u) gets row u -----------------------------------
        ok = tc_transform(f, pb, c, r, v, 0);
        if (!ok) break;

        // ---- exact top-k of the chunk, ties to the lowest index, records in index order ------------------
        // Fast path (k_eff <= 64): the k_eff-th largest of the 64 per-row maxima bounds the k_eff-th largest
        // coefficient from below; the coefficients at or above it (a few dozen) are listed in index order
        // and ranked exactly.  Everything compares integer magnitude keys (NaN and Inf are ordered like any
        // other bit pattern).  Too many candidates (tied chunks) or k_eff > 64: radix select over the tile.
        // `keep` collects, per row, which coefficients were kept: the inverse below takes them from there.
        DemoRecord *rec = a.payload + cr.te.rec_begin + cr.lc * (long long)k_eff;
        unsigned long long keep = 0ull;
        if (cr.valid) {
            write_own_row(X, r, v);
            unsigned *cand_key = hist, *cand_idx = hist + CAPT + 4;  // the histogram area doubles as the candidate lists
            bool use_radix = k_eff > S;
            if (!use_radix) {
                unsigned tkey = 0u;
#pragma unroll
                for (int j = 0; j < S; ++j) tkey = max(tkey, mag_key(v[j]));
                rowmask[2 * r] = 0u;
                rowmask[2 * r + 1] = 0u;
                misc[4 + r] = tkey;  // misc[4 .. 4 + 64): the maxima of the chunk's rows
                sb.sync();
                const unsigned okey = misc[4 + (r ^ 32)];
                const unsigned lo_all = __reduce_min_sync(0xffffffffu, min(tkey, okey));
                const unsigned hi_all = __reduce_max_sync(0xffffffffu, max(tkey, okey));
                if (hi_all == 0u) {
                    // every coefficient zero (a tile no gradient has touched yet): no selection needed, the
                    // tie rule gives the records 0 .. k_eff-1 (all in row 0, k_eff <= 64 here) with value 0
                    if (r < k_eff) {
                        DemoRecord rc;
                        rc.idx = r;
                        rc.val = 0.f;
                        rec[r] = rc;
                    }
                    keep = (r == 0) ? (k_eff >= 64 ? ~0ull : ((1ull << k_eff) - 1ull)) : 0ull;
                } else {
                const int b0 = 31 - __clz((lo_all ^ hi_all) | 0x8000u);  // >= 15
                unsigned lmin = lo_all & ~((2u << b0) - 1u);
#pragma unroll 1
                for (int bit = b0; bit >= 15; --bit) {
                    const unsigned cand = lmin | (1u << bit);
                    const unsigned cnt = __popc(__ballot_sync(0xffffffffu, tkey >= cand)) +
                                         __popc(__ballot_sync(0xffffffffu, okey >= cand));
                    lmin = (cnt >= (unsigned)k_eff) ? cand : lmin;
                }
                unsigned long long mask = 0ull;
#pragma unroll
                for (int j = 0; j < S; ++j) mask |= (unsigned long long)(mag_key(v[j]) >= lmin) << j;
                const unsigned cnt = (unsigned)__popcll(mask);
                const unsigned inc = warp_inclusive_scan(cnt, lane);
                if (lane == 31) misc[warp2] = inc;
                sb.sync();
                const unsigned n0 = misc[0], n_all = n0 + misc[1];
                use_radix = n_all > (unsigned)CAPT || n_all < (unsigned)k_eff;
                if (!use_radix) {
                    unsigned o = inc - cnt + (warp2 ? n0 : 0u);
                    while (mask) {
                        const int j = __ffsll((long long)mask) - 1;
                        mask &= mask - 1ull;
                        cand_key[o] = mag_key(X[r * XS + j]);
                        cand_idx[o] = (unsigned)(r * S + j);
                        ++o;
                    }
                    if (r < 4) cand_key[n_all + r] = 0u;  // pad for the vector loads
                    sb.sync();
                    // candidates r and r + 64 of the list (list order = index order)
                    unsigned selbits = 0u;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const unsigned me = (unsigned)(r + 64 * e);
                        if (me < n_all) {
                            const unsigned key = cand_key[me];
                            unsigned rank = 0;
                            const uint4 *keys4 = reinterpret_cast<const uint4 *>(cand_key);
                            for (unsigned c4 = 0; c4 < ((n_all + 3u) >> 2); ++c4) {
                                const uint4 k4 = keys4[c4];
                                const unsigned j0 = 4u * c4;
                                rank += (k4.x > key) || (k4.x == key && j0 < me);
                                rank += (k4.y > key) || (k4.y == key && j0 + 1u < me);
                                rank += (k4.z > key) || (k4.z == key && j0 + 2u < me);
                                rank += (k4.w > key) || (k4.w == key && j0 + 3u < me);
                            }
                            selbits |= (unsigned)(rank < (unsigned)k_eff) << (16 * e);
                        }
                    }
                    // positions: all kept among list entries 0..63 first (thread order), then among 64..127
                    const unsigned sinc = warp_inclusive_scan(selbits, lane);
                    if (lane == 31) misc[2 + warp2] = sinc;
                    sb.sync();
                    unsigned before = sinc - selbits + (warp2 ? misc[2] : 0u);
                    const unsigned tot = misc[2] + misc[3];
                    const unsigned pos_e[2] = {before & 0xffffu, (tot & 0xffffu) + (before >> 16)};
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        if ((selbits >> (16 * e)) & 1u) {
                            const unsigned idx = cand_idx[r + 64 * e];
                            DemoRecord rc;
                            rc.idx = (int)idx;
                            rc.val = X[(idx >> 6) * XS + (idx & (S - 1))];
                            rec[pos_e[e]] = rc;
                            atomicOr(&rowmask[2 * (idx >> 6) + ((idx >> 5) & 1u)], 1u << (idx & 31u));
                        }
                    }
                    sb.sync();
                    keep = ((unsigned long long)rowmask[2 * r + 1] << 32) | rowmask[2 * r];
                }
                }  // chunk not all zero
            }
            if (use_radix) {
                sb.sync();  // the coefficient tile is complete; the candidate path (if it ran) is done with its lists
                unsigned thr, need_eq;
                radix_select_tile<S, XS>(X, k_eff, hist, misc, &thr, &need_eq, r, sb);
                unsigned gt = 0, eq = 0;
#pragma unroll
                for (int j = 0; j < S; ++j) {
                    const unsigned key = mag_key(v[j]);
                    gt += key > thr;
                    eq += key == thr;
                }
                const unsigned packed = gt | (eq << 16);
                const unsigned inc = warp_inclusive_scan(packed, lane);
                sb.sync();  // the select's last reads of misc are done
                if (lane == 31) misc[warp2] = inc;
                sb.sync();
                unsigned before = inc - packed;
                if (warp2 == 1) before += misc[0];
                unsigned gb = before & 0xffffu, eb = before >> 16;
#pragma unroll
                for (int j = 0; j < S; ++j) {
                    const unsigned key = mag_key(v[j]);
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
                        DemoRecord rc;
                        rc.idx = r * S + j;
                        rc.val = v[j];
                        rec[pos] = rc;
                        keep |= 1ull << j;
                    }
                }
            }
        }
        pb.sync();  // both chunks are done with the tiles (coefficient tile, lists): they become operand space

        // ---- kept coefficients as a dense tile: row u of Q_sp (zero except the kept entries) --------------
#pragma unroll
        for (int j = 0; j < S; ++j) v[j] = ((keep >> j) & 1ull) ? v[j] : 0.f;
        // ---- R = P^T Q_sp P; momentum subtraction  m <- B - alpha R  (Section 2.1) -----------------------
        ok = tc_transform(f, pb, c, r, v, 1);
        if (!ok) break;
        if (cr.valid) {
#pragma unroll
            for (int j = 0; j < S; ++j) v[j] = fmaf(-a.alpha, v[j], b[j]);
            write_own_row(X, r, v);
            sb.sync();
#pragma unroll
            for (int it = 0; it < 16; ++it)
                *reinterpret_cast<float4 *>(m_tile + (size_t)sweep_row(it, r) * n1 + sweep_col(r)) =
                    *reinterpret_cast<const float4 *>(X + sweep_row(it, r) * XS + sweep_col(r));
        }
        pb.sync();  // the tiles are free for the next pair
    }
    if (!ok && f.pt == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
    tc_teardown(f);
}

__global__ void __launch_bounds__(TC_THREADS, 1) decode_tc_kernel(DemoDecodeArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    TcFrame f;
    tc_setup(f, smem_raw, a.C, false);
    const int c = f.pt >> 6, r = f.pt & 63;
    const SlotBarrier<PAIR_THREADS> pb{1 + f.g};
    const SlotBarrier<S> sb{1 + GROUPS + 2 * f.g + c};
    // aggregate tile of chunk c, and (count-normalised mean only) the senders per coordinate behind it
    float *St = reinterpret_cast<float *>(f.op + (c ? OFF_OP_LO : OFF_OP_HI));
    unsigned short *Cn = reinterpret_cast<unsigned short *>(St + S * XS);
    const bool counts = a.agg == 2;
    bool ok = true;

    const long long n_pairs = (a.n_chunks + 1) / 2;
    for (long long p = (long long)blockIdx.x * GROUPS + f.g; p < n_pairs; p += (long long)gridDim.x * GROUPS) {
        const ChunkRef cr = locate(a.entries, a.n_entries, a.n_chunks, 2 * p + c);
        const int k_eff = cr.te.k_eff;
        {
            // pull the next pair's parameter tiles into L2 while this pair is worked on
            const ChunkRef nx = locate(a.entries, a.n_entries, a.n_chunks, 2 * (p + (long long)gridDim.x * GROUPS) + c);
            if (nx.valid) {
                const char *nxp = reinterpret_cast<const char *>(a.x_ptrs[nx.te.tensor] + nx.tile_off) +
                                  (size_t)r * nx.te.n1 * sizeof(float);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nxp));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nxp + 128));
            }
        }
        float v[S];
        if (cr.valid) {
            float4 *row = reinterpret_cast<float4 *>(St + r * XS);
#pragma unroll
            for (int j4 = 0; j4 < S / 4; ++j4) row[j4] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (counts)
                for (int i = r; i < M / 2; i += S) reinterpret_cast<unsigned *>(Cn)[i] = 0u;
            sb.sync();
            // S = sum over workers in worker order (Decompress&Aggregate): indices are unique inside one
            // worker's chunk, a barrier per worker fixes the order of the additions
            const long long rec_off = cr.te.rec_begin + cr.lc * (long long)k_eff;
            for (int w = 0; w < a.W; ++w) {
                const DemoRecord *rec = a.payloads[w] + rec_off;
                for (int i = r; i < k_eff; i += S) {
                    const DemoRecord rc = rec[i];
                    if ((unsigned)rc.idx < (unsigned)M) {
                        const int at = (rc.idx >> 6) * XS + (rc.idx & (S - 1));
                        St[at] += rc.val;
                        if (counts) Cn[rc.idx] += 1;
                    } else {
                        atomicMax(a.status, DEMO_DEV_PAYLOAD);
                    }
                }
                sb.sync();
            }
            read_own_row(St, r, v);
            if (counts) {  // Sparse Top-k Averaging: sum / number of senders, 0/0 = 0
#pragma unroll
                for (int j = 0; j < S; ++j) {
                    const unsigned short n = Cn[r * S + j];
                    if (n > 1) v[j] = v[j] / (float)n;
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < S; ++j) v[j] = 0.f;
        }
        pb.sync();  // every row has been read: the tiles become operand space

        // ---- R = P^T S P, then  x <- x - lr (phi(R) + wd x), tile-wise and coalesced ---------------------
        ok = tc_transform(f, pb, c, r, v, 1);
        if (!ok) break;
        if (cr.valid) {
            write_own_row(St, r, v);
            sb.sync();
            float *x_tile = a.x_ptrs[cr.te.tensor] + cr.tile_off;
            const size_t n1 = (size_t)cr.te.n1;
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                float4 *xp = reinterpret_cast<float4 *>(x_tile + (size_t)sweep_row(it, r) * n1 + sweep_col(r));
                const float4 rv4 = *reinterpret_cast<const float4 *>(St + sweep_row(it, r) * XS + sweep_col(r));
                const float4 xv = *xp;
                const float rv[4] = {rv4.x, rv4.y, rv4.z, rv4.w};
                const float xe[4] = {xv.x, xv.y, xv.z, xv.w};
                float out[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float sg = a.phi ? rv[e] * a.agg_scale : (float)((rv[e] > 0.f) - (rv[e] < 0.f));
                    out[e] = fmaf(-a.lr, fmaf(a.wd, xe[e], sg), xe[e]);
                }
                *xp = make_float4(out[0], out[1], out[2], out[3]);
            }
        }
        pb.sync();  // the tiles are free for the next pair
    }
    if (!ok && f.pt == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
    tc_teardown(f);
}

template <typename K, typename A>
cudaError_t launch_tc(K kernel, const A &a, int sm_count, cudaStream_t stream)
{
    if (a.n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES);
    if (err != cudaSuccess) return err;
    const long long n_ctas = ((a.n_chunks + 1) / 2 + GROUPS - 1) / GROUPS;
    const long long grid = n_ctas < sm_count ? n_ctas : sm_count;  // one CTA per SM owns the tensor memory it needs
    kernel<<<(unsigned)grid, TC_THREADS, TC_SMEM_BYTES, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace

bool demo_tc_supported(int s) { return s == S; }

cudaError_t demo_launch_compress_tc(const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    return launch_tc(compress_tc_kernel, a, sm_count, stream);
}

cudaError_t demo_launch_decode_tc(const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    return launch_tc(decode_tc_kernel, a, sm_count, stream);
}
