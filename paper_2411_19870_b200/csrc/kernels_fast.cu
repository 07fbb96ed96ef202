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

#include <type_traits>

#include "demo_internal.h"
#include "fast_common.cuh"
#include "fast_dct.cuh"

namespace {

using namespace fastk;

constexpr int CAP = 128;                          // candidate capacity of the fast top-k
template <int S>
struct Cfg {
    static constexpr int XS = S + 4;  // row stride of the transpose tile: conflict-free scalar
                                      // column access and 128-bit row access
    static constexpr int NW = S / 32;
    static constexpr int LOG2S = (S == 64) ? 6 : 5;
};

// Bytes of the tile area of the compress kernel: the staged m and g tiles, or the padded transpose
// tile that later aliases them, whichever is larger.
template <int S, typename GT>
constexpr size_t compress_region_bytes()
{
    constexpr size_t stage = (size_t)S * S * (sizeof(float) + sizeof(GT));
    constexpr size_t xt = (size_t)S * Cfg<S>::XS * sizeof(float);
    return stage > xt ? stage : xt;
}

template <int S, typename GT>
constexpr size_t compress_slot_bytes()
{
    constexpr size_t raw = compress_region_bytes<S, GT>() + S * 4 + (CAP + 8) * 3 * 4 + 64 * 16 + 16 * 4 + 16;
    return (raw + 127) / 128 * 128;
}

template <int S, typename GT, bool TMAP, int THREADS>
__global__ void __launch_bounds__(THREADS, 512 / THREADS) compress_fast_kernel(DemoCompressArgs a)
{
    using C = Cfg<S>;
    constexpr int XS = C::XS, NW = C::NW, LOG2S = C::LOG2S;
    constexpr unsigned TILE_BYTES = S * S * sizeof(float) + S * S * sizeof(GT);
    constexpr int CAPW = CAP / NW;        // candidate capacity of one warp's list
    constexpr int CAPWP = CAPW + 4;       // list stride (padding for 128-bit key loads)
    constexpr int ITER = CAPW / 32;
    // wide candidate list (tiles of low rank or with a concentrated spectrum): one list per chunk in the part
    // of the staging area that the coefficient tile does not cover, 8 bytes per entry
    constexpr int WCAP_ROOM = (int)((compress_region_bytes<S, GT>() - (size_t)S * XS * sizeof(float)) / 8) - 4;
    constexpr int WCAP = WCAP_ROOM < 512 ? 128 : 512;
    static_assert(WCAP_ROOM >= 128, "the wide candidate list needs room behind the coefficient tile");

    extern __shared__ __align__(128) unsigned char smem_all[];
    const int slot = threadIdx.x / S;
    unsigned char *smem_raw = smem_all + (size_t)slot * compress_slot_bytes<S, GT>();
    const SlotBarrier<S> sb{slot + 1};
    // The staging area of the m and g tiles is reused as the transpose / coefficient / row-stage
    // tile X once column t has been consumed; B itself is not kept in shared memory: for the residual
    // the two tiles are fetched a second time (an L2 hit, issued behind the inverse transform).
    float *Ms = reinterpret_cast<float *>(smem_raw);             // [S*S]   m tile
    GT *Gs = reinterpret_cast<GT *>(Ms + S * S);                 // [S*S]   g tile
    float *X = Ms;                                               // [S*XS]  transpose / Q / T (aliases the tiles)
    float *tmax = reinterpret_cast<float *>(smem_raw + compress_region_bytes<S, GT>());  // [S]
    int *cand_idx = reinterpret_cast<int *>(tmax + S);           // [CAP]
    float *cand_val = reinterpret_cast<float *>(cand_idx + CAP + 8); // [CAP + 8]
    unsigned *cand_key = reinterpret_cast<unsigned *>(cand_val + CAP + 8);  // [CAP + 8]
    unsigned *hist = reinterpret_cast<unsigned *>(cand_idx);     // [256] aliases the candidate arrays
    int4 *recs4 = reinterpret_cast<int4 *>(cand_key + CAP + 8);  // [64] kept records, pre-decoded
    unsigned *misc = reinterpret_cast<unsigned *>(recs4 + 64);   // [16]
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(misc + 16);

    const int t = threadIdx.x % S, lane = t & 31, warp = t >> 5;
    const uint32_t bar = smem_u32(bar_mem);

    if (t == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();  // make the initialised barrier visible to the async proxy
    }
    __syncthreads();
    fence_proxy_async();
    bool failed = false;  // slot-uniform: a bounded wait of this slot expired

    EntryCursor cur;
    float *m_ptr = nullptr;
    const GT *g_ptr = nullptr;
    int cached_tensor = -1;
    unsigned phase = 0;
    const char *acquired = nullptr;  // the last tensor map made visible to the tensor-map proxy (thread 0 of the slot)

    // Locate the tile of chunk c (advances the tensor cursor; chunk ids only grow): tensor maps and box
    // coordinates for the TMA path, row t of the tile for the row-by-row path.
    struct TileRef {
        const char *tm_m, *tm_g;
        int x, y;
        const float *m_src;
        const GT *g_src;
    };
    auto locate = [&](long long c) {
        cur.seek(a.entries, a.n_entries, c);
        if (cur.te.tensor != cached_tensor) {
            cached_tensor = cur.te.tensor;
            m_ptr = a.m_ptrs[cached_tensor];
            g_ptr = reinterpret_cast<const GT *>(a.g_ptrs[cached_tensor]);
        }
        // chunks per tensor fit 31 bits (checked at init): 32-bit division
        const unsigned lc = (unsigned)(c - cur.te.chunk_begin);
        const unsigned k0 = lc / (unsigned)cur.te.c1;
        const int k1 = (int)(lc - k0 * (unsigned)cur.te.c1);
        TileRef r;
        r.tm_m = r.tm_g = nullptr;
        r.x = k1 * S;
        r.y = (int)k0 * S;
        r.m_src = nullptr;
        r.g_src = nullptr;
        if (TMAP) {
            r.tm_m = static_cast<const char *>(a.tmap_m) + (size_t)cached_tensor * TMAP_BYTES;
            r.tm_g = static_cast<const char *>(a.tmap_g) + (size_t)cached_tensor * TMAP_BYTES;
            if (t == 0 && r.tm_m != acquired) {  // first use of these maps by the issuing thread
                acquired = r.tm_m;
                tmap_acquire(r.tm_m);
                tmap_acquire(r.tm_g);
            }
        } else {
            const size_t off = ((size_t)k0 * S + t) * (size_t)cur.te.n1 + (size_t)k1 * S;
            r.m_src = m_ptr + off;
            r.g_src = g_ptr + off;
        }
        return r;
    };
    // Called right after a CTA-wide barrier that follows a fence.proxy.async of every thread.
    auto issue_loads = [&](const TileRef &r) {
        if (TMAP) {
            if (t == 0) {
                mbar_expect_tx(bar, TILE_BYTES);
                tma_load_2d(smem_u32(Ms), r.tm_m, r.x, r.y, bar);
                tma_load_2d(smem_u32(Gs), r.tm_g, r.x, r.y, bar);
            }
        } else {
            if (t == 0) mbar_expect_tx(bar, TILE_BYTES);
            bulk_g2s(smem_u32(Ms + t * S), r.m_src, S * sizeof(float), bar);
            bulk_g2s(smem_u32(Gs + t * S), r.g_src, S * sizeof(GT), bar);
        }
    };

    // chunk ids: CTA b, slot s, round r  ->  (r * gridDim.x + b) * NCH + s
    constexpr int NCH = THREADS / S;
    const long long stride = (long long)gridDim.x * NCH;
    long long c = (long long)blockIdx.x * NCH + slot;
    TileRef tile_cur, tile_next;
    if (c < a.n_chunks) {
        tile_cur = locate(c);
        issue_loads(tile_cur);
    }

    for (long long cb = (long long)blockIdx.x * NCH; cb < a.n_chunks; cb += stride, c += stride) {
        // all slots of the CTA start a chunk together; a slot whose wait expired takes the CTA down.
        // (Running the two halves of the slots half a chunk apart, or smaller CTAs, was measured
        // slower: the second instruction stream costs more than the overlap of phases gains.)
        if (__syncthreads_or(failed)) return;
        if (c >= a.n_chunks) continue;
        // the cursor points at chunk c (issue_loads(c) ran last)
        const DemoTensorEntry te = cur.te;
        const unsigned lc = (unsigned)(c - te.chunk_begin);
        const unsigned k0 = lc / (unsigned)te.c1;
        const int k1 = (int)(lc - k0 * (unsigned)te.c1);
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ m = m_ptr;
        const int k_eff = te.k_eff;
        DemoRecord *rec = a.payload + te.rec_begin + lc * (long long)k_eff;

        const bool arrived = mbar_wait_bounded(bar, phase);
        phase ^= 1u;
        if (!sb.sync_and(arrived)) {
            if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);  // give copies in flight one more bounded chance to land
            failed = true;
            continue;
        }
        // start pulling the next chunk's rows into L2 while this chunk is processed
        const long long nc = c + stride;
        if (nc < a.n_chunks) {
            tile_next = locate(nc);
            if (TMAP && t == 0) {
                tma_prefetch_2d(tile_next.tm_m, tile_next.x, tile_next.y);
                tma_prefetch_2d(tile_next.tm_g, tile_next.x, tile_next.y);
            }
        }

        // ---- momentum update on column t, then the two DCT passes --------------------------------
        // One copy of the unrolled transform serves both passes (the loop is kept rolled to halve the
        // instruction footprint): pass 0 runs down column t of B = beta*m + g and writes the
        // transpose tile, pass 1 runs along row t and leaves q[v] = Q[t][v] in registers.
        float q[S];
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            if (pass == 0) {
#pragma unroll
                for (int i = 0; i < S; ++i) q[i] = fmaf(a.beta, Ms[i * S + t], to_f32(Gs[i * S + t]));
                sb.sync();  // every thread has consumed its column of the staged tiles (X aliases them)
            } else {
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
            {
                float qi[S];
#pragma unroll
                for (int i = 0; i < S; ++i) qi[i] = q[i];
                fdct::dct2_packed<S, fdct::ScaleOrtho<S>>(qi, q);
                q[0] *= fdct::dc_scale<S>();
            }
            if (pass == 0) {
#pragma unroll
                for (int u = 0; u < S; ++u) X[u * XS + t] = q[u];
                sb.sync();
            }
        }

        // ---- top-k ------------------------------------------------------------------------------
        bool use_fallback = (k_eff > S);
        // A chunk whose coefficients are all zero (a gradient tile that was never touched, e.g. unused
        // embedding rows, on a momentum that is still zero) needs no selection: the tie rule gives it the
        // records 0 .. k_eff-1 with value 0.  Slot-uniform; found from the per-thread maxima.
        bool zero_chunk = false;
        unsigned n_cw = 0, off = 0;
        unsigned mlo = 0u, mhi = 0u;
        unsigned lmin_w = 0u;  // the bound L as a magnitude key (every candidate's key is >= it)
        if (!use_fallback) {
            // per-thread maximum magnitude: independent chains of 16 with 3-input max.  With S = 32 the two
            // chains stay apart (two maxima per thread): 64 groups again, so that the bound is still useful
            // at k_eff = 32.
            float tm = 0.f, tm2 = 0.f;
#pragma unroll
            for (int ch = 0; ch < S / 16; ++ch) {
                const int b0 = 16 * ch;
                float c = max3abs(q[b0], q[b0 + 1], q[b0 + 2]);
#pragma unroll
                for (int j = 3; j + 1 < 16; j += 2) c = max3f(c, fabsf(q[b0 + j]), fabsf(q[b0 + j + 1]));
                if (S == 32 && ch == 1)
                    tm2 = max3f(tm2, c, fabsf(q[b0 + 15]));
                else
                    tm = max3f(tm, c, fabsf(q[b0 + 15]));
            }
            // L = the k_eff-th largest of the 64 maxima.  Every warp holds all of them -- its own and the
            // partner warp's (S = 64), or its two per thread (S = 32) -- so that no second exchange is needed.
            const unsigned tkey = __float_as_uint(tm);
            unsigned *tk = reinterpret_cast<unsigned *>(tmax);
            if (NW > 1) {
                tk[t] = tkey;
                sb.sync();
            }
            unsigned lmin;
            {
                // bit-by-bit search, most significant first, for the largest L (low 15 mantissa bits zero)
                // that still has k_eff maxima at or above it: two ballots per step count them
                const unsigned okey = (NW > 1) ? tk[t ^ 32] : __float_as_uint(tm2);
                // the answer lies between the smallest and the largest maximum: their common leading
                // bits are settled, the search starts at the first bit where the two differ
                const unsigned both_min = min(tkey, okey), both_max = max(tkey, okey);
                const unsigned lo_all = __reduce_min_sync(0xffffffffu, both_min);
                const unsigned hi_all = __reduce_max_sync(0xffffffffu, both_max);
                zero_chunk = (hi_all == 0u);
                const int b0 = 31 - __clz((lo_all ^ hi_all) | 0x8000u);  // >= 15
                unsigned prefix = lo_all & ~((2u << b0) - 1u);
#pragma unroll 1
                for (int b = zero_chunk ? 14 : b0; b >= 15; --b) {
                    const unsigned cand = prefix | (1u << b);
                    const unsigned cnt = __popc(__ballot_sync(0xffffffffu, tkey >= cand)) +
                                         __popc(__ballot_sync(0xffffffffu, okey >= cand));
                    prefix = (cnt >= (unsigned)k_eff) ? cand : prefix;
                }
                lmin = prefix;
                lmin_w = prefix;
            }
            if (!zero_chunk) {
                const float L = __uint_as_float(lmin);
                // candidates: coefficients with magnitude >= L (at least k_eff of them exist).
                // |q| >= L  <=>  |q| > Lm with Lm the float just below L; the sign bit of Lm - |q| is
                // shifted into a bit mask (independent chains of 16).
                const float Lm = (L > 0.f) ? __uint_as_float(lmin - 1u) : -1.f;
                unsigned mc[S / 16];
    #pragma unroll
                for (int ch = 0; ch < S / 16; ++ch) {
                    unsigned mm = 0u;
    #pragma unroll
                    for (int j = 15; j >= 0; --j)
                        mm = __funnelshift_l(__float_as_uint(Lm - fabsf(q[16 * ch + j])), mm, 1);
                    mc[ch] = mm;
                }
                mlo = mc[0] | (mc[1] << 16);
                if (S == 64) mhi = mc[S / 16 - 2] | (mc[S / 16 - 1] << 16);
                // each warp compacts its candidates into its own list (rows of warp 0 precede rows of
                // warp 1, so the concatenation is in ascending index order)
                const unsigned cnt = __popc(mlo) + __popc(mhi);
                const unsigned inc = warp_inclusive_scan(cnt, lane);
                off = inc - cnt;
                n_cw = __shfl_sync(0xffffffffu, inc, 31);
                if (lane == 0) misc[warp] = n_cw;
            }
        }
        // stash the coefficients of row t (own row: no hazard with other threads)
        if (!zero_chunk) {
            float4 *row = reinterpret_cast<float4 *>(X + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(q[4 * v4], q[4 * v4 + 1], q[4 * v4 + 2], q[4 * v4 + 3]);
        }
        if (zero_chunk) {
            // k_eff <= S here: record i is (idx i, value 0); the row-stage list gets the same zeros
            if (t < k_eff) {
                DemoRecord r;
                r.idx = t;
                r.val = 0.f;
                rec[t] = r;
            }
            if (t < ((k_eff + 7) & ~7)) recs4[t] = make_int4(0, 0, 0, 0);
        } else if (!use_fallback) {
            const unsigned lbase = warp * CAPWP;
            if (n_cw <= CAPW) {
                unsigned o = lbase + off;
                unsigned long long mask = ((unsigned long long)mhi << 32) | mlo;
                while (mask) {
                    const int v = __ffsll((long long)mask) - 1;
                    mask &= mask - 1ull;
                    const float val = X[t * XS + v];
                    cand_idx[o] = t * S + v;
                    cand_val[o] = val;
                    cand_key[o] = mag_key(val);
                    ++o;
                }
                if (lane < 4) cand_key[lbase + n_cw + lane] = 0u;  // pad for the vector loads
            }
            sb.sync();
            unsigned n_w[NW], n_all = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                n_w[w] = misc[w];
                n_all += n_w[w];
                use_fallback = use_fallback || (n_w[w] > CAPW);
            }
            // Fewer than k_eff candidates cannot happen with finite data (the k_eff largest maxima are
            // candidates themselves); with NaN coefficients the comparisons above fail, and the select on
            // the integer keys, which orders every bit pattern, takes over.
            use_fallback = use_fallback || (n_all < (unsigned)k_eff);
            // Tiles of low rank (one active row or column: embedding and output-layer gradients) have row
            // maxima that bound the k-th coefficient loosely and list a few hundred candidates.  Lists of up
            // to WCAPW entries per warp, kept in the part of the staging area that the coefficient tile does
            // not cover, are ranked by a compact (rolled) version of the code below instead of sending the
            // whole chunk through the radix select.
            bool wide = false;
            if constexpr (NW > 1) {
                // Too many candidates even for the wide list: a finer partition bounds the k_eff-th coefficient
                // more tightly -- the maxima of the 256 quarter rows and of the 256 quarter columns (a tile with
                // a few active columns has rows that all look alike, and the other way round).  Taken from the
                // stashed tile, only on this path; the candidates are then listed again under the largest bound.
                if (n_all > (unsigned)WCAP) {
                    unsigned rk[4], ck[4];
                    const float4 *row4 = reinterpret_cast<const float4 *>(X + t * XS);
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        unsigned m = 0u;
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            const float4 f = row4[4 * g + v4];
                            m = max(max(m, mag_key(f.x)), max(mag_key(f.y), max(mag_key(f.z), mag_key(f.w))));
                        }
                        rk[g] = m;
                    }
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        unsigned m = 0u;
#pragma unroll 4
                        for (int u = 0; u < 16; ++u) m = max(m, mag_key(X[(16 * g + u) * XS + t]));
                        ck[g] = m;
                    }
                    // every warp needs all 512 maxima: its own and, through shared memory, the partner warp's
                    unsigned *gq = reinterpret_cast<unsigned *>(smem_raw + (size_t)S * XS * sizeof(float));  // [8][64]
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        gq[g * 64 + t] = rk[g];
                        gq[(4 + g) * 64 + t] = ck[g];
                    }
                    sb.sync();
                    unsigned prk[4], pck[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        prk[g] = gq[g * 64 + (t ^ 32)];
                        pck[g] = gq[(4 + g) * 64 + (t ^ 32)];
                    }
                    // the k_eff-th largest of 256 keys (four of this thread, four of its partner), low 15 bits zero
                    auto kth_of_256 = [&](const unsigned (&own)[4], const unsigned (&oth)[4]) -> unsigned {
                        unsigned lo = 0xffffffffu, hi = 0u;
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            lo = min(lo, min(own[g], oth[g]));
                            hi = max(hi, max(own[g], oth[g]));
                        }
                        lo = __reduce_min_sync(0xffffffffu, lo);
                        hi = __reduce_max_sync(0xffffffffu, hi);
                        const int c0 = 31 - __clz((lo ^ hi) | 0x8000u);
                        unsigned pre = lo & ~((2u << c0) - 1u);
#pragma unroll 1
                        for (int b = c0; b >= 15; --b) {
                            const unsigned cand = pre | (1u << b);
                            unsigned cnt = 0;
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                cnt += __popc(__ballot_sync(0xffffffffu, own[g] >= cand)) +
                                       __popc(__ballot_sync(0xffffffffu, oth[g] >= cand));
                            pre = (cnt >= (unsigned)k_eff) ? cand : pre;
                        }
                        return pre;
                    };
                    const unsigned l2 = max(kth_of_256(rk, prk), kth_of_256(ck, pck));
                    if (l2 > lmin_w) {  // slot-uniform
                        lmin_w = l2;
                        unsigned long long mask = 0ull;
#pragma unroll 4
                        for (int v = 0; v < S; ++v) mask |= (unsigned long long)(mag_key(X[t * XS + v]) >= l2) << v;
                        mlo = (unsigned)mask;
                        mhi = (unsigned)(mask >> 32);
                        const unsigned cnt = __popc(mlo) + __popc(mhi);
                        const unsigned inc = warp_inclusive_scan(cnt, lane);
                        off = inc - cnt;
                        n_cw = __shfl_sync(0xffffffffu, inc, 31);
                        if (lane == 0) misc[warp] = n_cw;
                        sb.sync();
                        n_all = 0;
#pragma unroll
                        for (int w = 0; w < NW; ++w) {
                            n_w[w] = misc[w];
                            n_all += n_w[w];
                        }
                    }
                }
            }
            if (use_fallback && n_all >= (unsigned)k_eff && n_all <= (unsigned)WCAP) {
                wide = true;
                use_fallback = false;
            }
            if (wide) {
                unsigned *wkey = reinterpret_cast<unsigned *>(smem_raw + (size_t)S * XS * sizeof(float));  // [WCAP + 4]
                unsigned *widx = wkey + WCAP + 4;
                {
                    // one list in index order: the rows of warp 0, then the rows of warp 1
                    unsigned o = ((NW > 1 && warp == 1) ? n_w[0] : 0u) + off;
                    unsigned long long mask = ((unsigned long long)mhi << 32) | mlo;
                    while (mask) {
                        const int v = __ffsll((long long)mask) - 1;
                        mask &= mask - 1ull;
                        widx[o] = t * S + v;
                        wkey[o] = mag_key(X[t * XS + v]);
                        ++o;
                    }
                }
                sb.sync();
                // Every warp takes the whole list into registers (WK keys per lane) and finds the k_eff-th
                // largest key by the same bit-by-bit ballot search as for the bound -- no exchange between the
                // warps.  Entries above it are kept, entries equal to it in index order until k_eff are
                // reached; the record position of a kept entry is the number of kept entries before it.  Every
                // warp forms the running counts over the whole list and writes the groups that are its own.
                auto wide_select = [&](auto wk_tag) {
                    constexpr int WK = decltype(wk_tag)::value;
                    unsigned keys[WK];
                    unsigned hi = 0u;
#pragma unroll
                    for (int j = 0; j < WK; ++j) {
                        const unsigned i = (unsigned)j * 32u + lane;
                        keys[j] = (i < n_all) ? wkey[i] : 0u;  // absent entries: 0, below every candidate
                        hi = max(hi, keys[j]);
                    }
                    hi = __reduce_max_sync(0xffffffffu, hi);
                    // every entry is >= lmin_w (> 0 here): the bits above the first one where lmin_w and the
                    // largest key differ are settled
                    const int wb0 = 31 - __clz((lmin_w ^ hi) | 1u);
                    unsigned thr = lmin_w & ~((2u << wb0) - 1u);
#pragma unroll 1
                    for (int b = wb0; b >= 0; --b) {
                        const unsigned cand = thr | (1u << b);
                        unsigned cnt = 0;
#pragma unroll
                        for (int j = 0; j < WK; ++j) cnt += __popc(__ballot_sync(0xffffffffu, keys[j] >= cand));
                        thr = (cnt >= (unsigned)k_eff) ? cand : thr;
                    }
                    unsigned n_gt = 0;
#pragma unroll
                    for (int j = 0; j < WK; ++j) n_gt += __popc(__ballot_sync(0xffffffffu, keys[j] > thr));
                    const unsigned need_eq = (unsigned)k_eff - n_gt;  // >= 1
                    unsigned gt_before = 0, eq_before = 0;
                    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
                    for (int j = 0; j < WK; ++j) {
                        const unsigned key = keys[j];
                        const unsigned gtb = __ballot_sync(0xffffffffu, key > thr);
                        const unsigned eqb = __ballot_sync(0xffffffffu, key == thr);
                        if ((j % NW) == warp) {
                            const unsigned e = eq_before + __popc(eqb & lt);
                            if ((key > thr) || (key == thr && e < need_eq)) {
                                const unsigned pos = gt_before + __popc(gtb & lt) + min(e, need_eq);
                                DemoRecord r;
                                r.idx = (int)widx[j * 32 + lane];
                                const int v = r.idx & (S - 1);
                                const int uo = (r.idx >> LOG2S) * XS;
                                r.val = X[uo + v];
                                rec[pos] = r;
                                recs4[pos] = make_int4(uo, v * S, __float_as_int(a.alpha * r.val), 0);
                                if ((int)pos == k_eff - 1)
                                    for (int pp = k_eff; pp < ((k_eff + 7) & ~7); ++pp) recs4[pp] = make_int4(uo, 0, 0, 0);
                            }
                        }
                        gt_before += __popc(gtb);
                        eq_before += __popc(eqb);
                    }
                };
                if (WCAP <= 128 || n_all <= 128u)
                    wide_select(std::integral_constant<int, 4>{});
                else
                    wide_select(std::integral_constant<int, WCAP / 32>{});
            } else if (!use_fallback) {
                // rank among all candidates by magnitude only.  If exactly k_eff candidates have
                // fewer than k_eff larger ones, no tie straddles the threshold and that set is the
                // answer; otherwise the count is redone with the index tie-break.
                bool sel[ITER];
                unsigned pre[ITER];
#pragma unroll
                for (int it = 0; it < ITER; ++it) {
                    const unsigned li = it * 32 + lane;  // position in this warp's list
                    sel[it] = false;
                    if (it * 32 < (int)n_cw) {  // warp-uniform
                        const unsigned key = (li < n_cw) ? cand_key[lbase + li] : 0xffffffffu;
                        unsigned rank = 0;
#pragma unroll
                        for (int w = 0; w < NW; ++w) {
                            const uint4 *keys4 = reinterpret_cast<const uint4 *>(cand_key + w * CAPWP);
                            const unsigned n4 = (n_w[w] + 3u) >> 2;
                            for (unsigned c4 = 0; c4 < n4; ++c4) {
                                const uint4 k4 = keys4[c4];
                                rank += (k4.x > key) + (k4.y > key) + (k4.z > key) + (k4.w > key);
                            }
                        }
                        sel[it] = (li < n_cw) && rank < (unsigned)k_eff;
                    }
                    const unsigned bal = __ballot_sync(0xffffffffu, sel[it]);
                    pre[it] = __popc(bal & ((1u << lane) - 1u));
                    if (lane == 0) misc[4 + warp * ITER + it] = __popc(bal);
                }
                sb.sync();
                unsigned total = 0;
#pragma unroll
                for (int g = 0; g < ITER * NW; ++g) total += misc[4 + g];
                if (total != (unsigned)k_eff) {  // block-uniform: equal magnitudes straddle the threshold
                    sb.sync();
#pragma unroll
                    for (int it = 0; it < ITER; ++it) {  // (rare path: inner loops stay rolled)
                        const unsigned li = it * 32 + lane;
                        sel[it] = false;
                        if (li < n_cw) {
                            const unsigned key = cand_key[lbase + li];
                            unsigned rank = 0;
#pragma unroll
                            for (int w = 0; w < NW; ++w)
#pragma unroll 1
                                for (unsigned c2 = 0; c2 < n_w[w]; ++c2) {
                                    const unsigned k2 = cand_key[w * CAPWP + c2];
                                    const bool earlier = (w < warp) || (w == warp && c2 < li);
                                    rank += (k2 > key) || (k2 == key && earlier);
                                }
                            sel[it] = rank < (unsigned)k_eff;
                        }
                        const unsigned bal = __ballot_sync(0xffffffffu, sel[it]);
                        pre[it] = __popc(bal & ((1u << lane) - 1u));
                        if (lane == 0) misc[4 + warp * ITER + it] = __popc(bal);
                    }
                    sb.sync();
                }
#pragma unroll
                for (int it = 0; it < ITER; ++it) {
                    if (sel[it]) {
                        unsigned pos = pre[it];
                        for (int g = 0; g < warp * ITER + it; ++g) pos += misc[4 + g];
                        DemoRecord r;
                        r.idx = cand_idx[lbase + it * 32 + lane];
                        r.val = cand_val[lbase + it * 32 + lane];
                        rec[pos] = r;
                        const int v = r.idx & (S - 1);  // k_eff <= S <= 64 on this path
                        const int uo = (r.idx >> LOG2S) * XS;
                        recs4[pos] = make_int4(uo, v * S, __float_as_int(a.alpha * r.val), 0);
                        if ((int)pos == k_eff - 1)
                            for (int pp = k_eff; pp < ((k_eff + 7) & ~7); ++pp) recs4[pp] = make_int4(uo, 0, 0, 0);
                    }
                }
            }
        }
        if (use_fallback) {
            sb.sync();  // coefficient tile complete in X
            unsigned thr, need_eq;
            radix_select_tile<S, XS>(X, k_eff, hist, misc, &thr, &need_eq, t, sb);
            unsigned gt = 0, eq = 0;
#pragma unroll 1
            for (int v = 0; v < S; ++v) {
                const unsigned key = mag_key(X[t * XS + v]);
                gt += key > thr;
                eq += key == thr;
            }
            const unsigned packed = gt | (eq << 16);
            const unsigned inc = warp_inclusive_scan(packed, lane);
            sb.sync();  // radix_select_tile's last reads of misc are done
            if (lane == 31) misc[warp] = inc;
            sb.sync();
            unsigned before = inc - packed;
#pragma unroll
            for (int w = 0; w < NW; ++w)
                if (w < warp) before += misc[w];
            unsigned gb = before & 0xffffu, eb = before >> 16;
#pragma unroll 1
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
                    if (k_eff <= 64) {
                        recs4[pos] = make_int4(t * XS, v * S, __float_as_int(a.alpha * val), 0);
                        if ((int)pos == k_eff - 1)
                            for (int pp = k_eff; pp < ((k_eff + 7) & ~7); ++pp) recs4[pp] = make_int4(t * XS, 0, 0, 0);
                    }
                }
            }
        }
        sb.sync();  // records complete (shared list and global payload); X is free

        // ---- residual: row stage of the inverse from the k_eff records, sparse ------------------
        {
            float4 *row = reinterpret_cast<float4 *>(X + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        sb.sync();
        {
            // T[u][t] = sum over kept (u, v) of val * C[v][t]; the basis is read through L1 (all CTAs
            // of the SM share the same 4*S*S bytes), coalesced across the warp
            const float *Ct = a.C + t;
            float acc = 0.f;
            int cur_u = -1;
            if (k_eff <= 64) {
                // the list is padded to a multiple of eight with zero-valued records of the last row;
                // eight records and their cosines are fetched ahead of the dependent accumulation
                cur_u = recs4[0].x;
                for (int r0 = 0; r0 < k_eff; r0 += 8) {
                    int4 rc[8];
                    float cv[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) rc[j] = recs4[r0 + j];
#pragma unroll
                    for (int j = 0; j < 8; ++j) cv[j] = __ldg(Ct + rc[j].y);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const bool chg = rc[j].x != cur_u;
                        if (chg) X[cur_u + t] = acc;
                        acc = chg ? 0.f : acc;
                        cur_u = rc[j].x;
                        acc = fmaf(__int_as_float(rc[j].z), cv[j], acc);
                    }
                }
            } else {
                for (int r = 0; r < k_eff; ++r) {
                    const DemoRecord rc = rec[r];
                    const int u = (rc.idx >> LOG2S) * XS, v = rc.idx & (S - 1);
                    if (u != cur_u) {
                        if (cur_u >= 0) X[cur_u + t] = acc;
                        acc = 0.f;
                        cur_u = u;
                    }
                    acc = fmaf(a.alpha * rc.val, __ldg(Ct + v * S), acc);
                }
            }
            if (cur_u >= 0) X[cur_u + t] = acc;
        }
        // column t of T was written by this thread only: no barrier needed before reading it back
        {
            float r[S];
#pragma unroll
            for (int u = 0; u < S; ++u) r[u] = X[u * XS + t];
            // X is dead: fetch the m and g tiles again (they were read moments ago, so this is an L2
            // hit) while the inverse transform runs, and rebuild B = beta*m + g for the residual
            fence_proxy_async();
            sb.sync();
            issue_loads(tile_cur);
            {
                float ri[S];
                r[0] *= fdct::dc_scale<S>();
#pragma unroll
                for (int i = 0; i < S; ++i) ri[i] = r[i];
                fdct::dct3_packed<S, fdct::ScaleOrtho<S>>(ri, r);
            }
            const bool again = mbar_wait_bounded(bar, phase);
            phase ^= 1u;
            if (!sb.sync_and(again)) {
                if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
                mbar_wait_bounded(bar, phase ^ 1u);
                failed = true;
                continue;
            }
#pragma unroll
            for (int i = 0; i < S; ++i)
                m[base + (size_t)i * te.n1 + t] = fmaf(a.beta, Ms[i * S + t], to_f32(Gs[i * S + t])) - r[i];
        }
        fence_proxy_async();  // order this thread's shared-memory accesses before the async-proxy writes
        sb.sync();      // the staging area is free again
        if (nc < a.n_chunks) {
            tile_cur = tile_next;
            issue_loads(tile_cur);
        }
    }
}

// Bytes of one decode slot: the tile, the mbarrier and -- for the count-normalised mean -- one
// 16-bit sender count per coordinate.
constexpr int STAGE_RECORDS = 512;  // records staged per batch of the scatter (sixteen workers at k <= 32)
template <int S>
__host__ __device__ constexpr size_t decode_slot_bytes(bool counts)
{
    return ((size_t)S * Cfg<S>::XS * 4 + 16 + 2 * STAGE_RECORDS * sizeof(DemoRecord) + (counts ? (size_t)S * S * 2 : 0) + 127) /
           128 * 128;
}

// SIGNS: the parameter-server form -- sign(R) goes out as int8 per element, the parameters are neither read
// nor written (a separate instantiation, so that the update kernel keeps its size).
// WIDE: the instantiation for fan-ins above one staging batch (sixteen workers at k <= 32): every further batch of a
// chunk's workers is requested, like the first, while the scatter works on the batch before it.
template <int S, bool TMAP, int THREADS, bool SIGNS = false, bool WIDE = false>
__global__ void __launch_bounds__(THREADS, 512 / THREADS) decode_fast_kernel(DemoDecodeArgs a)
{
    using C = Cfg<S>;
    constexpr int XS = C::XS, NCH = THREADS / S;
    constexpr int M = S * S;
    extern __shared__ __align__(128) unsigned char smem_all[];
    const int slot = threadIdx.x / S;
    const bool counts = a.agg == 2;
    unsigned char *smem_raw = smem_all + (size_t)slot * decode_slot_bytes<S>(counts);
    const SlotBarrier<S> sb{slot + 1};
    // One tile per slot: the aggregate S, then the row-stage output, and -- once column t has been
    // read back into registers -- the staging area of the x tile, fetched behind the second transform.
    float *St = reinterpret_cast<float *>(smem_raw);  // [S*XS]
    float *Xt = St;                                   // [S*S] (aliases St)
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(St + S * XS);
    DemoRecord *stage_all = reinterpret_cast<DemoRecord *>(bar_mem + 2);    // [2][STAGE_RECORDS] records of a batch of workers
    unsigned short *Cn = reinterpret_cast<unsigned short *>(stage_all + 2 * STAGE_RECORDS);  // [S*S] senders per coordinate (agg == 2)

    const int t = threadIdx.x % S;
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
    bool failed = false;
    const char *acquired = nullptr;
    const unsigned lr_bits = __float_as_uint(a.lr);
    const float decay = 1.f - a.lr * a.wd;
    const float neg_lr_scale = -a.lr * a.agg_scale;

    // The records of a chunk's first batch of workers (up to STAGE_RECORDS records) are copied into one of two
    // staging buffers by asynchronous copies issued a whole chunk ahead, so that the payload reads of the W
    // workers -- W small pieces from W buffers -- never stand in front of the scatter.  One copy group per chunk.
    auto stage_ahead = [&](int buf, long long chunk) {
        cur.seek(a.entries, a.n_entries, chunk);
        const int k_n = cur.te.k_eff;
        if (k_n <= 64) {
            const long long off_n = cur.te.rec_begin + (chunk - cur.te.chunk_begin) * (long long)k_n;
            const int sh = (k_n > 32) ? 6 : 5;
            DemoRecord *dst = stage_all + buf * STAGE_RECORDS;
#pragma unroll
            for (int i = 0; i < STAGE_RECORDS / S; ++i) {
                const int r = i * S + t, wl = r >> sh, j = r & ((1 << sh) - 1);
                if (wl < a.W && j < k_n)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst + r)),
                                 "l"(a.payloads[wl] + off_n + j)
                                 : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // (WIDE) a further batch of the same chunk: workers w_first .. of the chunk whose records start at off_n
    auto stage_batch = [&](int buf, int k_n, long long off_n, int w_first) {
        const int sh = (k_n > 32) ? 6 : 5;
        DemoRecord *dst = stage_all + buf * STAGE_RECORDS;
#pragma unroll
        for (int i = 0; i < STAGE_RECORDS / S; ++i) {
            const int r = i * S + t, wl = w_first + (r >> sh), j = r & ((1 << sh) - 1);
            if (wl < a.W && j < k_n)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst + r)),
                             "l"(a.payloads[wl] + off_n + j)
                             : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    const long long stride = (long long)gridDim.x * NCH;
    long long c = (long long)blockIdx.x * NCH + slot;
    int buf = 0;
    if (c < a.n_chunks) stage_ahead(0, c);
    for (long long cb = (long long)blockIdx.x * NCH; cb < a.n_chunks; cb += stride, c += stride) {
        if (__syncthreads_or(failed)) break;  // all slots start a chunk together (shared instruction stream)
        if (c >= a.n_chunks) continue;
        cur.seek(a.entries, a.n_entries, c);
        const DemoTensorEntry te = cur.te;
        if (te.tensor != cached_tensor) {
            cached_tensor = te.tensor;
            x_ptr = a.x_ptrs[cached_tensor];
        }
        const unsigned lc = (unsigned)(c - te.chunk_begin);
        const unsigned k0 = lc / (unsigned)te.c1;
        const int k1 = (int)(lc - k0 * (unsigned)te.c1);
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ x = x_ptr;
        const int k_eff = te.k_eff;
        const long long rec_off = te.rec_begin + lc * (long long)k_eff;
        if (TMAP && !SIGNS && t == 0) {
            const char *tm_x = static_cast<const char *>(a.tmap_x) + (size_t)te.tensor * TMAP_BYTES;
            if (tm_x != acquired) {  // first use of this tensor's map by the issuing thread
                acquired = tm_x;
                tmap_acquire(tm_x);
            }
            tma_prefetch_2d(tm_x, k1 * S, (int)k0 * S);
        }

        {
            float4 *row = reinterpret_cast<float4 *>(St + t * XS);
#pragma unroll
            for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (counts)
                for (int v = 0; v < S; ++v) Cn[t * S + v] = 0;
        }
        auto stage_next_chunk = [&](int into) {  // (the cursor moves on; this chunk's table entry is in `te`)
            if (c + stride < a.n_chunks)
                stage_ahead(into, c + stride);
            else
                asm volatile("cp.async.commit_group;" ::: "memory");
        };
        DemoRecord *stage = stage_all + buf * STAGE_RECORDS;
        if (!WIDE || k_eff > 64) {
            // next chunk's records on their way
            stage_next_chunk(buf ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");  // this chunk's copies have landed
            buf ^= 1;
        }
        // S = sum over workers in worker order (Decompress&Aggregate).
        if (k_eff <= 64) {
            // Every warp owns the 32 rows of the tile its threads cleared and will transform (rows 32 w .. 32 w + 31
            // for warp w of the slot).  The records of up to sixteen workers (512 records) are staged in shared
            // memory with one round of global loads; then every warp walks the staged workers in order, reads ALL
            // records of a worker (lane j: record j, and j + 32 where k > 32) and adds those that fall into its rows.
            // A coordinate is only ever touched by one warp, so the order of the additions -- worker after worker,
            // hence bit-reproducible -- needs nothing but warp-level synchronisation.
            const int lane = t & 31, warp = t >> 5;
            const int sh = (k_eff > 32) ? 6 : 5;          // a worker's records take 32 or 64 staging entries
            const int wb = STAGE_RECORDS >> sh;           // workers per batch: 16 or 8
            for (int w0 = 0; w0 < a.W; w0 += wb) {
                if (WIDE) {
                    // both warps are done with the previous batch (between chunks the barrier at the end of a chunk
                    // has seen to that): its buffer takes the batch after this one -- of this chunk's workers or,
                    // behind the last, the first batch of the slot's next chunk
                    if (w0 > 0) sb.sync();
                    if (w0 + wb < a.W)
                        stage_batch(buf ^ 1, k_eff, rec_off, w0 + wb);
                    else
                        stage_next_chunk(buf ^ 1);
                    asm volatile("cp.async.wait_group 1;" ::: "memory");  // this batch's copies have landed
                    stage = stage_all + buf * STAGE_RECORDS;
                    buf ^= 1;
                } else if (w0 > 0) {  // further batches of a large fan-in: fetched on the spot
                    sb.sync();  // the previous batch has been consumed by both warps
#pragma unroll 1
                    for (int r = t; r < STAGE_RECORDS; r += S) {
                        const int wl = r >> sh, j = r & ((1 << sh) - 1);
                        if (w0 + wl < a.W && j < k_eff) stage[r] = a.payloads[w0 + wl][rec_off + j];
                    }
                }
                sb.sync();  // staged records visible (also orders the clearing of the tile before the first additions)
                const int nw = min(wb, a.W - w0);
                // (the next worker's record is read before this worker's addition, so that only the addition itself
                // lies between two warp barriers)
                const bool two = k_eff > 32;
                DemoRecord nx0 = stage[lane], nx1 = stage[two ? lane + 32 : lane];
#pragma unroll 1
                for (int wl = 0; wl < nw; ++wl) {
                    const DemoRecord rc0 = nx0, rc1 = nx1;
                    if (wl + 1 < nw) {
                        nx0 = stage[((wl + 1) << sh) + lane];
                        if (two) nx1 = stage[((wl + 1) << sh) + lane + 32];
                    }
                    if (lane < k_eff) {
                        if ((unsigned)rc0.idx < (unsigned)M) {
                            if ((rc0.idx >> (C::LOG2S + 5)) == warp) {
                                St[(rc0.idx >> C::LOG2S) * XS + (rc0.idx & (S - 1))] += rc0.val;
                                if (counts) Cn[rc0.idx] += 1;
                            }
                        } else {
                            atomicMax(a.status, DEMO_DEV_PAYLOAD);
                        }
                    }
                    if (two && lane + 32 < k_eff) {
                        if ((unsigned)rc1.idx < (unsigned)M) {
                            if ((rc1.idx >> (C::LOG2S + 5)) == warp) {
                                St[(rc1.idx >> C::LOG2S) * XS + (rc1.idx & (S - 1))] += rc1.val;
                                if (counts) Cn[rc1.idx] += 1;
                            }
                        } else {
                            atomicMax(a.status, DEMO_DEV_PAYLOAD);
                        }
                    }
                    __syncwarp();
                }
            }
        } else {
            // k > 64: a thread's records may fall into any row; a barrier per worker fixes the order of additions.
            // Records are fetched eight workers ahead so that one memory latency covers eight workers.
            sb.sync();
            for (int kb = 0; kb < k_eff; kb += S) {
                const bool mine = kb + t < k_eff;
                for (int w0 = 0; w0 < a.W; w0 += 8) {
                    DemoRecord r[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (mine && w0 + j < a.W) r[j] = a.payloads[w0 + j][rec_off + kb + t];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (w0 + j < a.W) {
                            if (mine) {
                                if ((unsigned)r[j].idx < (unsigned)M) {
                                    St[(r[j].idx >> C::LOG2S) * XS + (r[j].idx & (S - 1))] += r[j].val;
                                    if (counts) Cn[r[j].idx] += 1;
                                } else {
                                    atomicMax(a.status, DEMO_DEV_PAYLOAD);
                                }
                            }
                            sb.sync();
                        }
                    }
                }
            }
        }
        if (counts) {  // Sparse Top-k Averaging: sum / number of senders, 0/0 = 0 (row t is this thread's)
            for (int v = 0; v < S; ++v) {
                const unsigned short n = Cn[t * S + v];
                if (n > 1) St[t * XS + v] = St[t * XS + v] / (float)n;
            }
        }
        // Two inverse passes through one copy of the unrolled transform (rolled loop): pass 0 along
        // row t in place, pass 1 down column t; the x tile is fetched while pass 1 computes.
        float r[S];
        bool arrived = true;
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            if (pass == 0) {
                const float4 *row = reinterpret_cast<const float4 *>(St + t * XS);
#pragma unroll
                for (int v4 = 0; v4 < S / 4; ++v4) {
                    const float4 f = row[v4];
                    r[4 * v4 + 0] = f.x;
                    r[4 * v4 + 1] = f.y;
                    r[4 * v4 + 2] = f.z;
                    r[4 * v4 + 3] = f.w;
                }
            } else {
#pragma unroll
                for (int u = 0; u < S; ++u) r[u] = St[u * XS + t];
                fence_proxy_async();
                sb.sync();  // the tile is dead: stage x into it
                if (SIGNS) {
                    // nothing to stage
                } else if (TMAP) {
                    if (t == 0) {
                        mbar_expect_tx(bar, S * S * sizeof(float));
                        tma_load_2d(smem_u32(Xt), static_cast<const char *>(a.tmap_x) + (size_t)te.tensor * TMAP_BYTES,
                                    k1 * S, (int)k0 * S, bar);
                    }
                } else {
                    if (t == 0) mbar_expect_tx(bar, S * S * sizeof(float));
                    bulk_g2s(smem_u32(Xt + t * S), x + base + (size_t)t * te.n1, S * sizeof(float), bar);
                }
            }
            {
                // inverse transform: the DCT-IV blocks and the butterfly cascade with two sums per instruction
                // (same results as the scalar form)
                float w[S], y[S];
                fdct::static_for<0, S>([&](auto i) { w[decltype(i)::value] = r[fdct::core_index<S>(decltype(i)::value)]; });
                fdct::dct_core_ortho_paired<S>(w, y);
                fdct::dct3_post_paired<S>(y, r);
            }
            if (pass == 0) {
                float4 *row = reinterpret_cast<float4 *>(St + t * XS);
#pragma unroll
                for (int v4 = 0; v4 < S / 4; ++v4)
                    row[v4] = make_float4(r[4 * v4], r[4 * v4 + 1], r[4 * v4 + 2], r[4 * v4 + 3]);
                sb.sync();
            } else if (!SIGNS) {
                arrived = mbar_wait_bounded(bar, phase);
                phase ^= 1u;
            }
        }
        if constexpr (SIGNS) {
            signed char *__restrict__ sg = a.sign_ptrs[te.tensor];
#pragma unroll
            for (int i = 0; i < S; ++i) sg[base + (size_t)i * te.n1 + t] = (signed char)((r[i] > 0.f) - (r[i] < 0.f));
            sb.sync();  // the tile is free again
            continue;
        }
        if (!sb.sync_and(arrived)) {
            if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);
            failed = true;
            continue;
        }
        // sign and update:  x - lr (sign(R) + wd x) = x (1 - lr wd) - lr sign(R); -lr sign(R) is lr with
        // its sign flipped where R > 0, and zero where R == 0
#pragma unroll
        for (int i = 0; i < S; ++i) {
            const float rv = r[i];
            float stepv = __uint_as_float(lr_bits ^ (~__float_as_uint(rv) & 0x80000000u));
            stepv = (rv == 0.f) ? 0.f : stepv;
            if (a.phi) stepv = rv * neg_lr_scale;  // phi = identity: -lr * R (R / W for the mean)
            x[base + (size_t)i * te.n1 + t] = fmaf(Xt[i * S + t], decay, stepv);
        }
        sb.sync();  // the tile is free again
    }
    asm volatile("cp.async.wait_all;" ::: "memory");  // no copy of this thread may outlive the CTA's shared memory
}

// CTA sizes: the compress kernel runs best with all eight slots of an SM in one CTA (one shared
// instruction stream); fp32 gradients need a larger staging area, so fewer slots fit.  The decode
// kernel, whose code fits the instruction cache, runs best with every slot in a CTA of its own
// (8192 x 8192 case: 103 us with 64-thread CTAs, 108 us with 128, 114 us with 256).
template <int S, typename GT>
constexpr int compress_threads()
{
    return (S == 64) ? ((sizeof(GT) == 2) ? 512 : 256) : 256;
}
constexpr int DECODE_THREADS = 64;

// Persistent launch: CTAs of `threads` threads (threads / S slots), as many as fit the device, each
// striding over groups of chunks.
template <typename K>
cudaError_t launch(K kernel, int threads, int nch, size_t smem, long long n_chunks, int sm_count, cudaStream_t stream,
                   const void *args)
{
    if (n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    int per_sm = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const long long groups = (n_chunks + nch - 1) / nch;
    long long grid = (long long)sm_count * per_sm;
    if (grid > groups) grid = groups;
    void *params[] = {const_cast<void *>(args)};
    return cudaLaunchKernel((const void *)kernel, dim3((unsigned)grid), dim3(threads), params, smem, stream);
}

template <int S, typename GT>
cudaError_t launch_compress(const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    constexpr int TH = compress_threads<S, GT>();
    constexpr int NCH = TH / S;
    const size_t smem = compress_slot_bytes<S, GT>() * NCH;
    if (a.tmap_m != nullptr && a.tmap_g != nullptr)
        return launch(compress_fast_kernel<S, GT, true, TH>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
    return launch(compress_fast_kernel<S, GT, false, TH>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
}

template <int S>
cudaError_t launch_decode(const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    constexpr int TH = DECODE_THREADS;
    constexpr int NCH = TH / S;
    const size_t smem = decode_slot_bytes<S>(a.agg == 2) * NCH;
    if (a.sign_ptrs != nullptr)
        return launch(decode_fast_kernel<S, false, TH, true>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
    if (a.tmap_x != nullptr) {
        if (a.W > 16)  // more than one staging batch at k <= 32
            return launch(decode_fast_kernel<S, true, TH, false, true>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
        return launch(decode_fast_kernel<S, true, TH>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
    }
    return launch(decode_fast_kernel<S, false, TH>, TH, NCH, smem, a.n_chunks, sm_count, stream, &a);
}

// One CTA arms an mbarrier with a transaction count that no copy will ever satisfy and waits for it
// with the same bounded wait the production kernels use.
__global__ void wait_selftest_kernel(int *status, long long limit_cycles)
{
    __shared__ __align__(8) unsigned long long bar_mem;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_expect_tx(bar, 16);  // 16 bytes that never arrive
    const bool arrived = mbar_wait_bounded(bar, 0, limit_cycles);
    if (!__syncthreads_and(arrived) && threadIdx.x == 0) atomicMax(status, DEMO_DEV_TIMEOUT);
}

}  // namespace

cudaError_t demo_launch_wait_selftest(int *status, long long limit_cycles, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 64, 0, stream>>>(status, limit_cycles);
    return cudaGetLastError();
}

bool demo_fast_supported(int s) { return s == 128 || s == 64 || s == 32; }

cudaError_t demo_launch_compress_fast(int s, const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    if (s == 128) return demo_launch_compress_fast128(a, sm_count, stream);
    if (s == 64) {
#ifndef DEMO_OLD64
        if (a.tmap_m != nullptr && a.tmap_g != nullptr) return demo_launch_compress_fast64(a, sm_count, stream);
#endif
        return a.grad_bf16 ? launch_compress<64, __nv_bfloat16>(a, sm_count, stream)
                           : launch_compress<64, float>(a, sm_count, stream);
    }
    if (s == 32)
        return a.grad_bf16 ? launch_compress<32, __nv_bfloat16>(a, sm_count, stream)
                           : launch_compress<32, float>(a, sm_count, stream);
    return cudaErrorInvalidValue;
}

cudaError_t demo_launch_decode_fast(int s, const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    if (s == 128) return demo_launch_decode_fast128(a, sm_count, stream);
    if (s == 64) return launch_decode<64>(a, sm_count, stream);
    if (s == 32) return launch_decode<32>(a, sm_count, stream);
    return cudaErrorInvalidValue;
}
