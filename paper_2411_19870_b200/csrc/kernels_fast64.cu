// Compress kernel for 2-D tensors with chunk size 64 (the paper's main configuration): Algorithm 1 worker
// side / CompressChunks, fused per chunk -- momentum update, 2-D DCT-II, exact top-k, momentum
// subtraction.  64 threads (a "slot") own one 64 x 64 chunk; thread t works on column t, then row t.
//
// What shapes this kernel is its instruction footprint.  A register-resident 64-point transform is
// ~10 KB of straight-line code; three copies (two forward passes, one inverse) plus fully unrolled
// tile reads do not fit the SM's instruction cache, and warps that sit at different places of such
// a stream starve on instruction fetch.  Here the hot loop is kept near 30 KB so that every slot can
// run on its own, and the phases of different chunks (tile wait, transform, selection, store burst)
// overlap on the SM's pipes instead of following one another:
//   * the three transform passes of a chunk go through ONE copy of the multiplications (the DCT-IV blocks
//     that DCT-II and DCT-III share, fast_dct.cuh) inside a rolled loop; only the butterfly cascades differ;
//   * B = beta*m + g is parked in tensor memory (one tcgen05.st of the thread's column) and read back for
//     the residual, instead of fetching and recombining the two tiles a second time;
//   * the next chunk's tiles are requested as soon as the transpose tile is dead, so they land behind
//     the inverse transform and the store burst of the current chunk;
//   * everything rare (tied or degenerate chunks, tiles of low rank, k > 64) lives in one out-of-line
//     routine that works from the coefficient tile in shared memory.
// Every wait on an mbarrier is bounded: on expiry the slot records DEMO_DEV_TIMEOUT and stops.
#include <cuda_bf16.h>

#include <type_traits>

#include "demo_internal.h"
#include "fast_common.cuh"
#include "fast_dct.cuh"

namespace {

using namespace fastk;

constexpr int S = 64;
constexpr int XS = S + 4;     // row stride of the transpose tile: conflict-free column access, 128-bit row access
constexpr int LOG2S = 6;
constexpr int CAP = 128;      // candidate capacity of the fast top-k (two lists of 64)
constexpr int CAPW = CAP / 2;
constexpr int CAPWP = CAPW + 4;
constexpr int WCAP = 512;     // capacity of the wide candidate list (out-of-line path)
constexpr int TMEM_COLS_PER_GROUP = 64;  // one column block per four warps (two slots)
constexpr int ROW_AHEAD = 8;              // entries of the row-stage list fetched ahead

// Tile area of a slot:  [0, 64*68*4)  the padded transpose / coefficient / row-stage tile X; its first 16 KB double as
// the landing area of the m tile and as the source of the TMA store of the new momentum;  behind it the landing
// area of the g tile, which between its two uses holds the lists of the selection: wide candidate list, big-k list, and -- at its
// end -- the row-stage list.
constexpr size_t TILE_X_BYTES = (size_t)S * XS * sizeof(float);
template <typename GT>
constexpr size_t region_bytes()
{
    constexpr size_t g_bytes = (size_t)S * S * sizeof(GT);
    constexpr size_t lists = (size_t)(WCAP + 4) * 8 + 256 * 8 + 65 * 16;  // wide list + big-k list + row-stage list
    static_assert(lists <= g_bytes, "the selection's lists live in the g landing area");
    return TILE_X_BYTES + g_bytes;
}
template <typename GT>
constexpr size_t slot_bytes()
{
    constexpr size_t raw = region_bytes<GT>() + S * 4 + (CAP + 8) * 3 * 4 + 16 * 4 + 16;
    return (raw + 127) / 128 * 128;
}

// Shared memory of one slot.
struct SlotMem {
    unsigned char *raw;
    float *X;            // [S*XS] transpose / coefficient / row-stage tile (aliases the staged tiles)
    float *tmax;         // [S]
    int *cand_idx;       // [CAP + 8]
    float *cand_val;     // [CAP + 8]
    unsigned *cand_key;  // [CAP + 8]
    unsigned *hist;      // [256] aliases the candidate arrays
    int4 *recs4;         // [65] kept records, pre-decoded for the row stage; entry 64 is always padding
    unsigned *misc;      // [16]
    unsigned *wkey;      // [WCAP + 4] wide list, behind the tile
    unsigned *widx;      // [WCAP + 4]
    uint2 *rbig;         // [256] kept records for 64 < k <= 256: (row << 16 | column, alpha * value), behind the wide list
};

// ------------------------------------------------------------------------------------------------
// Out-of-line selection for the chunks the in-line path does not take: more than 64 candidates in a
// warp's list (tiles of low rank or with a concentrated spectrum, tied or degenerate chunks), fewer
// candidates than k (NaN coefficients) or k > 64 (for 64 < k <= 256 the bound comes from step 2 alone).  Works from the coefficient tile in X (row t is
// this thread's), writes the records to `rec` and, for k <= 64, the pre-decoded list for the row stage.
//   1. wide list: up to WCAP candidates under the bound `lmin` (the k-th largest of the 64 row maxima),
//      every warp takes the whole list into registers and finds the exact k-th largest key by a
//      bit-by-bit ballot search;
//   2. if the list overflows: a tighter bound from the 256 quarter-row and the 256 quarter-column
//      maxima, then 1. again;
//   3. otherwise an exact 4 x 8-bit radix select over the whole tile.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void select_slow(const SlotMem sm, int k_eff, DemoRecord *rec, float alpha, int t, int bar_id,
                                         unsigned lmin_w, bool bound_valid, bool qdom)
{
    const SlotBarrier<S> sb{bar_id};
    const int lane = t & 31, warp = t >> 5;
    float *X = sm.X;
    unsigned *misc = sm.misc;
    int4 *recs4 = sm.recs4;
    sb.sync();  // the coefficient tile is complete; the in-line path is done with its lists

    bool done = false;
    if (k_eff <= 256) {  // (the finer bound below needs at least k groups: 256 quarter rows / quarter columns)
        unsigned long long mask = 0ull;
        unsigned off = 0, n_all = 0xffffffffu;
        auto count_under = [&](unsigned bound) {
            mask = 0ull;
#pragma unroll 4
            for (int v = 0; v < S; ++v) mask |= (unsigned long long)(mag_key(X[t * XS + v]) >= bound) << v;
            const unsigned cnt = (unsigned)__popcll(mask);
            const unsigned inc = warp_inclusive_scan(cnt, lane);
            sb.sync();  // earlier readers of misc are done
            if (lane == 31) misc[warp] = inc;
            sb.sync();
            const unsigned n0 = misc[0];
            n_all = n0 + misc[1];
            off = inc - cnt + (warp ? n0 : 0u);
        };
        if (bound_valid)
            count_under(lmin_w);
        else
            lmin_w = 0u;  // k > 64: the row maxima give no bound, the finer partition does
        if (n_all > (unsigned)WCAP) {
            // tighter bound: the k_eff-th largest of the 256 quarter-row maxima and of the 256 quarter-column maxima
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
            // (the quarter-column maxima matter for tiles with a few active columns; with k > 64, where this is the
            // ordinary path of every chunk, the quarter rows alone give the bound)
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                unsigned m = 0u;
                if (bound_valid) {
#pragma unroll 4
                    for (int u = 0; u < 16; ++u) m = max(m, mag_key(X[(16 * g + u) * XS + t]));
                }
                ck[g] = m;
            }
            unsigned *gq = sm.wkey;  // [8][64], behind the tile
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
            unsigned l2 = kth_of_256(rk, prk);
            if (bound_valid) l2 = max(l2, kth_of_256(ck, pck));
            sb.sync();  // gq is read; the wide list may overwrite it
            if (l2 > lmin_w || !bound_valid) {
                lmin_w = l2;
                count_under(lmin_w);
            }
        }
        if (n_all >= (unsigned)k_eff && n_all <= (unsigned)WCAP) {
            unsigned *wkey = sm.wkey, *widx = sm.widx;
            {
                unsigned o = off;
                while (mask) {
                    const int v = __ffsll((long long)mask) - 1;
                    mask &= mask - 1ull;
                    widx[o] = t * S + v;
                    wkey[o] = mag_key(X[t * XS + v]);
                    ++o;
                }
            }
            sb.sync();
            auto wide_select = [&](auto wk_tag) {
                constexpr int WK = decltype(wk_tag)::value;
                unsigned keys[WK];
                unsigned hi = 0u;
#pragma unroll
                for (int j = 0; j < WK; ++j) {
                    const unsigned i = (unsigned)j * 32u + lane;
                    keys[j] = (i < n_all) ? wkey[i] : 0u;
                    hi = max(hi, keys[j]);
                }
                hi = __reduce_max_sync(0xffffffffu, hi);
                const int wb0 = 31 - __clz((lmin_w ^ hi) | 1u);
                unsigned thr = lmin_w & ~((2u << wb0) - 1u);
                unsigned n_ge = n_all;  // every entry is >= the bound >= thr; the search stops at exactly k_eff
#pragma unroll 1
                for (int b = wb0; b >= 0 && n_ge != (unsigned)k_eff; --b) {
                    const unsigned cand = thr | (1u << b);
                    unsigned cnt = 0;
#pragma unroll
                    for (int j = 0; j < WK; ++j) cnt += __popc(__ballot_sync(0xffffffffu, keys[j] >= cand));
                    if (cnt >= (unsigned)k_eff) {
                        thr = cand;
                        n_ge = cnt;
                    }
                }
                unsigned n_gt = 0;
#pragma unroll
                for (int j = 0; j < WK; ++j) n_gt += __popc(__ballot_sync(0xffffffffu, keys[j] > thr));
                const unsigned need_eq = (unsigned)k_eff - n_gt;
                unsigned gt_before = 0, eq_before = 0;
                const unsigned lt = (1u << lane) - 1u;
#pragma unroll
                for (int j = 0; j < WK; ++j) {
                    const unsigned key = keys[j];
                    const unsigned gtb = __ballot_sync(0xffffffffu, key > thr);
                    const unsigned eqb = __ballot_sync(0xffffffffu, key == thr);
                    if ((j & 1) == warp) {
                        const unsigned e = eq_before + __popc(eqb & lt);
                        if ((key > thr) || (key == thr && e < need_eq)) {
                            const unsigned pos = gt_before + __popc(gtb & lt) + min(e, need_eq);
                            DemoRecord r;
                            r.idx = (int)widx[j * 32 + lane];
                            const int v = r.idx & (S - 1);
                            const int uo = (r.idx >> LOG2S) * XS;
                            r.val = X[uo + v];
                            rec[pos] = r;
                            if (qdom)  // transform-domain momentum: what stays of a transmitted coefficient
                                X[uo + v] = fmaf(-alpha, r.val, r.val);
                            else if (k_eff <= 64)
                                recs4[pos] = make_int4(uo, v * S, __float_as_int(alpha * r.val), 0);
                            else
                                sm.rbig[pos] = make_uint2(((unsigned)r.idx >> LOG2S) << 16 | (unsigned)v, __float_as_uint(alpha * r.val));
                        }
                    }
                    gt_before += __popc(gtb);
                    eq_before += __popc(eqb);
                }
            };
            if (n_all <= 128u)
                wide_select(std::integral_constant<int, 4>{});
            else
                wide_select(std::integral_constant<int, WCAP / 32>{});
            done = true;
        }
    }
    if (!done) {
        unsigned thr, need_eq;
        sb.sync();
        radix_select_tile<S, XS>(X, k_eff, sm.hist, misc, &thr, &need_eq, t, sb);
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
        if (warp == 1) before += misc[0];
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
                if (qdom)
                    X[t * XS + v] = fmaf(-alpha, val, val);
                else if (k_eff <= 64)
                    recs4[pos] = make_int4(t * XS, v * S, __float_as_int(alpha * val), 0);
                else if (k_eff <= 256)
                    sm.rbig[pos] = make_uint2((unsigned)t << 16 | (unsigned)v, __float_as_uint(alpha * val));
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Last step of the in-line selection: the k_eff largest of the n_all candidates (all >= the bound `lmin_w`, at most
// 32 * NK of them; list 0 holds the first n_w0 in ascending index order, list 1 the rest).  Every warp takes all
// candidates into registers, NK keys per lane in list order, and searches bit by bit, from the first bit where the
// bound and the largest key differ, for a threshold with exactly k_eff keys at or above it; the search stops as
// soon as one is found.  If it runs out of bits, equal keys straddle the k_eff-th place: keys above the threshold
// are kept, keys equal to it in index order until k_eff are reached.  A kept candidate's place among the records
// is the number of kept candidates before it; warp w writes the records of the key groups w, w + 2, ...
// ------------------------------------------------------------------------------------------------
template <int NK, bool QDOM>
__device__ __forceinline__ void ballot_select(const SlotMem &sm, unsigned n_w0, unsigned n_all, unsigned lmin_w, int k_eff,
                                              DemoRecord *rec, float alpha, int lane, int warp)
{
    static_assert(NK == 2 || NK == 4, "two or four keys per lane");
    auto list_pos = [&](unsigned i) { return i < n_w0 ? i : i - n_w0 + (unsigned)CAPWP; };
    unsigned keys[NK];
    unsigned hi = 0u;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        const unsigned i = (unsigned)j * 32u + lane;
        keys[j] = (i < n_all) ? sm.cand_key[list_pos(i)] : 0u;
        hi = max(hi, keys[j]);
    }
    hi = __reduce_max_sync(0xffffffffu, hi);
    const int wb0 = 31 - __clz((lmin_w ^ hi) | 1u);
    unsigned thr = lmin_w & ~((2u << wb0) - 1u);
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
#pragma unroll 1
    for (int jj = 0; jj < NK / 2; ++jj) {  // (rolled: one copy of the record write)
        const bool second = (jj != 0);     // key groups 2, 3 (NK = 4 only)
        const unsigned key = second ? (warp ? keys[NK - 1] : keys[NK - 2]) : (warp ? keys[1] : keys[0]);
        const unsigned gb = second ? (warp ? gtb[NK - 1] : gtb[NK - 2]) : (warp ? gtb[1] : gtb[0]);
        const unsigned eb = second ? (warp ? eqb[NK - 1] : eqb[NK - 2]) : (warp ? eqb[1] : eqb[0]);
        // kept / equal candidates in the key groups before this one
        unsigned gt_before = warp ? __popc(second ? gtb[NK - 2] : gtb[0]) : 0u;
        unsigned eq_before = warp ? __popc(second ? eqb[NK - 2] : eqb[0]) : 0u;
        if (second) {
            gt_before += __popc(gtb[0]) + __popc(gtb[1]);
            eq_before += __popc(eqb[0]) + __popc(eqb[1]);
        }
        const unsigned e = eq_before + __popc(eb & lt);
        if ((key > thr) || (key == thr && e < need_eq)) {
            const unsigned pos = gt_before + __popc(gb & lt) + min(e, need_eq);
            const unsigned li = list_pos((unsigned)(2 * jj + warp) * 32u + lane);
            DemoRecord r;
            r.idx = sm.cand_idx[li];
            r.val = sm.cand_val[li];
            rec[pos] = r;
            if (QDOM)  // what stays of a transmitted coefficient: q - alpha q
                sm.X[(r.idx >> LOG2S) * XS + (r.idx & (S - 1))] = fmaf(-alpha, r.val, r.val);
            else
                sm.recs4[pos] = make_int4((r.idx >> LOG2S) * XS, (r.idx & (S - 1)) * S, __float_as_int(alpha * r.val), 0);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Exact top-k of one chunk (Section 2.1 "Top-k Sparsification"): thread t holds the coefficients q[v] = Q[t][v] of
// row t.  Writes the k_eff records in ascending index order to `rec`; ends before the barrier that makes them
// visible.  QDOM = false (momentum kept in the spatial domain): also leaves the pre-decoded row-stage list and the
// tile X cleared for the row stage.  QDOM = true (momentum kept in the transform domain): leaves in X the
// coefficient tile with every transmitted coefficient q replaced by q - alpha q.
// ------------------------------------------------------------------------------------------------
template <bool QDOM>
__device__ __forceinline__ void select_chunk(const SlotMem &sm, float (&q)[S], int k_eff, DemoRecord *rec, float alpha,
                                             int t, const SlotBarrier<S> &sb, int bar_id, int pad_row)
{
    float *X = sm.X;
    float *tmax = sm.tmax;
    int *cand_idx = sm.cand_idx;
    float *cand_val = sm.cand_val;
    unsigned *cand_key = sm.cand_key;
    int4 *recs4 = sm.recs4;
    unsigned *misc = sm.misc;
    const int lane = t & 31, warp = t >> 5;
    // the row-stage tile starts from zero; every thread clears its own row once it is done with it
    auto zero_row = [&]() {
        if (QDOM) return;  // (the transform-domain kernel keeps the coefficient tile: it is its output)
        float4 *row = reinterpret_cast<float4 *>(X + t * XS);
#pragma unroll
        for (int v4 = 0; v4 < S / 4; ++v4) row[v4] = make_float4(0.f, 0.f, 0.f, 0.f);
    };
    // The stash of row t.  With the momentum in the spatial domain it is written in the transform core's own order
    // (position p holds coefficient core_index(p)): the registers of a 128-bit store are then neighbours in the
    // core's output, as the pairs of the inverse cascade are, and no register moves are needed to satisfy both.
    constexpr bool CORE_STASH = !QDOM;
    auto stash_row = [&](auto core_order) {
        float4 *row = reinterpret_cast<float4 *>(X + t * XS);
        fdct::static_for<0, S / 4>([&](auto i) {
            constexpr int v4 = decltype(i)::value;
            constexpr bool CO = decltype(core_order)::value;
            constexpr int i0 = CO ? fdct::core_index<S>(4 * v4) : 4 * v4, i1 = CO ? fdct::core_index<S>(4 * v4 + 1) : 4 * v4 + 1;
            constexpr int i2 = CO ? fdct::core_index<S>(4 * v4 + 2) : 4 * v4 + 2, i3 = CO ? fdct::core_index<S>(4 * v4 + 3) : 4 * v4 + 3;
            row[v4] = make_float4(q[i0], q[i1], q[i2], q[i3]);
        });
    };
    // position of coefficient v in a stash kept in core order: v = (2j + 1) << s sits at (32 >> s) + j, v = 0 at 0
    auto stash_pos = [](int v) {
        if (!CORE_STASH) return v;
        const int sft = __ffs(v | S) - 1;
        return ((S / 2) >> sft) + (v >> (sft + 1));
    };
    // ---- exact top-k (Section 2.1 "Top-k Sparsification") -------------------------------
    if (!QDOM) {
        recs4[t] = make_int4(pad_row, 0, 0, 0);  // list padding (ordered before the record writes by the barriers below)
        if (t == 0) recs4[64] = make_int4(pad_row, 0, 0, 0);
    }
    bool slow = (k_eff > S);
    bool bound_valid = false;
    bool zero_chunk = false;
    unsigned n_cw = 0, off = 0, mlo = 0u, mhi = 0u, lmin_w = 0u;
    if (!slow) {
        // per-thread maximum magnitude (independent chains of 16, 3-input max)
        float tm = 0.f;
#pragma unroll
        for (int ch = 0; ch < S / 16; ++ch) {
            const int b0 = 16 * ch;
            float cm = max3abs(q[b0], q[b0 + 1], q[b0 + 2]);
#pragma unroll
            for (int j = 3; j + 1 < 16; j += 2) cm = max3f(cm, fabsf(q[b0 + j]), fabsf(q[b0 + j + 1]));
            tm = max3f(tm, cm, fabsf(q[b0 + 15]));
        }
        // L = the k_eff-th largest of the 64 row maxima (low 15 mantissa bits cleared): a lower bound of
        // the k_eff-th largest coefficient.  Every warp holds all 64 keys, two ballots per step count them.
        const unsigned tkey = __float_as_uint(tm);
        unsigned *tk = reinterpret_cast<unsigned *>(tmax);
        tk[t] = tkey;
        sb.sync();
        const unsigned okey = tk[t ^ 32];
        const unsigned lo_all = __reduce_min_sync(0xffffffffu, min(tkey, okey));
        const unsigned hi_all = __reduce_max_sync(0xffffffffu, max(tkey, okey));
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
        lmin_w = prefix;
        bound_valid = true;
        if (!zero_chunk) {
            // candidates: |q| >= L  <=>  |q| > Lm (the float just below L); the sign bit of Lm - |q|
            // is funnel-shifted into a bit mask (independent chains of 16)
            const float L = __uint_as_float(lmin_w);
            const float Lm = (L > 0.f) ? __uint_as_float(lmin_w - 1u) : -1.f;
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
            mhi = mc[2] | (mc[3] << 16);
            const unsigned cnt = __popc(mlo) + __popc(mhi);
            const unsigned inc = warp_inclusive_scan(cnt, lane);
            off = inc - cnt;
            n_cw = __shfl_sync(0xffffffffu, inc, 31);
            if (lane == 0) misc[warp] = n_cw;
        }
    }
    if (zero_chunk) {
        // all coefficients zero: the tie rule gives the records 0 .. k_eff-1 with value 0
        if (t < k_eff) {
            DemoRecord r;
            r.idx = t;
            r.val = 0.f;
            rec[t] = r;
        }
        if (!QDOM && t < k_eff) recs4[t] = make_int4(0, 0, 0, 0);
        zero_row();
        if (QDOM) stash_row(std::false_type{});  // (all zero; the tile is the kernel's output)
    } else {
        // stash the coefficients of row t (own row: no hazard with other threads)
        stash_row(std::integral_constant<bool, CORE_STASH>{});
        if (!slow) {
            const unsigned lbase = warp * CAPWP;
            if (n_cw <= CAPW) {
                // each warp compacts its candidates into its own list (rows of warp 0 precede rows of
                // warp 1, so the concatenation is in ascending index order)
                unsigned o = lbase + off;
                unsigned long long mask = ((unsigned long long)mhi << 32) | mlo;
                while (mask) {
                    const int v = __ffsll((long long)mask) - 1;
                    mask &= mask - 1ull;
                    const float val = X[t * XS + stash_pos(v)];
                    cand_idx[o] = t * S + v;
                    cand_val[o] = val;
                    cand_key[o] = mag_key(val);
                    ++o;
                }
            }
            sb.sync();
            const unsigned n_w0 = misc[0], n_w1 = misc[1];
            // more than a list holds, or fewer candidates than k_eff (NaN coefficients fail the float
            // comparisons above): the out-of-line selection takes over
            slow = (n_w0 > (unsigned)CAPW) || (n_w1 > (unsigned)CAPW) || (n_w0 + n_w1 < (unsigned)k_eff);
            if (!slow) {
                zero_row();  // row t of the stash was read by this thread only
                // the two lists, read one behind the other, are in ascending index order
                if (n_w0 + n_w1 <= 64u)
                    ballot_select<2, QDOM>(sm, n_w0, n_w0 + n_w1, lmin_w, k_eff, rec, alpha, lane, warp);
                else
                    ballot_select<4, QDOM>(sm, n_w0, n_w0 + n_w1, lmin_w, k_eff, rec, alpha, lane, warp);
            }
        }
        if (slow) {
            if (CORE_STASH) stash_row(std::false_type{});  // the out-of-line selection reads the tile in index order
            select_slow(sm, k_eff, rec, alpha, t, bar_id, lmin_w, bound_valid, QDOM);
            sb.sync();  // every thread is done with the coefficient tile
            zero_row();
        }
    }
}

// QDOM = false: the momentum buffers hold the momentum itself (the contract of demo_compress).  QDOM = true (opt-in,
// demo_set_momentum_domain): they hold its chunk-wise DCT, tile by tile and transposed (element (r, c) of a tile
// is coefficient (c, r)): the step is then Q = beta*Qm + DCT(g), top-k, Qm <- Q - alpha*Q_kept -- one forward
// transform of the gradient, no inverse transform, no row stage.
template <typename GT, int THREADS, bool QDOM>
__global__ void __launch_bounds__(THREADS, 512 / THREADS) compress64_kernel(DemoCompressArgs a)
{
    constexpr int NCH = THREADS / S;
    constexpr int NGROUPS = (THREADS + 127) / 128;                   // groups of four warps
    constexpr int TMEM_COLS = NGROUPS * TMEM_COLS_PER_GROUP < 32 ? 32 : NGROUPS * TMEM_COLS_PER_GROUP;
    static_assert((TMEM_COLS & (TMEM_COLS - 1)) == 0, "tensor-memory allocations are powers of two");
    constexpr unsigned TILE_BYTES = S * S * sizeof(float) + S * S * sizeof(GT);

    extern __shared__ __align__(128) unsigned char smem_all[];
    const int slot = threadIdx.x / S;
    SlotMem sm;
    sm.raw = smem_all + (size_t)slot * slot_bytes<GT>();
    float *Ms = reinterpret_cast<float *>(sm.raw);             // [S*S] m tile
    GT *Gs = reinterpret_cast<GT *>(sm.raw + TILE_X_BYTES);    // [S*S] g tile
    sm.X = Ms;
    sm.wkey = reinterpret_cast<unsigned *>(sm.raw + TILE_X_BYTES);
    sm.widx = sm.wkey + WCAP + 4;
    sm.rbig = reinterpret_cast<uint2 *>(sm.widx + WCAP + 4);
    sm.tmax = reinterpret_cast<float *>(sm.raw + region_bytes<GT>());
    sm.cand_idx = reinterpret_cast<int *>(sm.tmax + S);
    sm.cand_val = reinterpret_cast<float *>(sm.cand_idx + CAP + 8);
    sm.cand_key = reinterpret_cast<unsigned *>(sm.cand_val + CAP + 8);
    sm.hist = reinterpret_cast<unsigned *>(sm.cand_idx);
    sm.recs4 = reinterpret_cast<int4 *>(sm.raw + region_bytes<GT>()) - 65;
    sm.misc = reinterpret_cast<unsigned *>(sm.cand_key + CAP + 8);
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(sm.misc + 16);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_all + (size_t)NCH * slot_bytes<GT>());
    float *X = sm.X;
    int4 *recs4 = sm.recs4;

    // "row" of the padding entries of the row-stage list: the scratch line tmax[0..S) seen from X
    constexpr int PAD_ROW = (int)(region_bytes<GT>() / sizeof(float));
    const int t = threadIdx.x % S;
    const int hw_warp = threadIdx.x >> 5;
    const SlotBarrier<S> sb{slot + 1};
    const uint32_t bar = smem_u32(bar_mem);

    if (t == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();
    }
    if (hw_warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    fence_proxy_async();
    const uint32_t tmem_base = *tmem_slot;
    // this thread's lane of tensor memory (a warp reaches the 32 lanes of its quadrant) and its slot's columns
    const uint32_t taddr = tmem_base + ((uint32_t)((hw_warp & 3) * 32) << 16) + (uint32_t)((hw_warp >> 2) * TMEM_COLS_PER_GROUP);

    EntryCursor cur;
    const char *acquired = nullptr;  // (thread 0) the last tensor map made visible to the tensor-map proxy
    unsigned phase = 0;

    // Tile of chunk c: tensor maps and box coordinates (the cursor is moved to c; chunk ids only grow).
    struct TileRef {
        const char *tm_m, *tm_g;
        int x, y;
    };
    auto locate = [&](long long c) {
        cur.seek(a.entries, a.n_entries, c);
        const unsigned lc = (unsigned)(c - cur.te.chunk_begin);
        const unsigned k0 = lc / (unsigned)cur.te.c1;
        const int k1 = (int)(lc - k0 * (unsigned)cur.te.c1);
        TileRef r;
        r.x = k1 * S;
        r.y = (int)k0 * S;
        r.tm_m = static_cast<const char *>(a.tmap_m) + (size_t)cur.te.tensor * TMAP_BYTES;
        r.tm_g = static_cast<const char *>(a.tmap_g) + (size_t)cur.te.tensor * TMAP_BYTES;
        return r;
    };
    // (thread 0) request the tiles of a chunk; a tensor map that this thread has not used yet is acquired first
    auto issue_loads = [&](const TileRef &r) {
        if (r.tm_m != acquired) {
            acquired = r.tm_m;
            tmap_acquire(r.tm_m);
            tmap_acquire(r.tm_g);
        }
        mbar_expect_tx(bar, TILE_BYTES);
        tma_load_2d(smem_u32(Ms), r.tm_m, r.x, r.y, bar);
        tma_load_2d(smem_u32(Gs), r.tm_g, r.x, r.y, bar);
    };

    const long long stride = (long long)gridDim.x * NCH;
    long long c = (long long)blockIdx.x * NCH + slot;
    TileRef next{};
    if (c < a.n_chunks) {
        next = locate(c);
        if (t == 0) issue_loads(next);
    }

    for (; c < a.n_chunks; c += stride) {
        // the cursor points at chunk c (its loads were issued last)
        const int k_eff = cur.te.k_eff;
        DemoRecord *rec = a.payload + cur.te.rec_begin + (c - cur.te.chunk_begin) * (long long)k_eff;

        // every thread waits for the tiles by itself; whether the wait expired is settled for the whole slot
        // at the first barrier of pass 0 (no barrier lies in between)
        const bool arrived = mbar_wait_bounded(bar, phase);
        phase ^= 1u;
        bool dead = false;
        // where this chunk's tile goes back to and where the next one comes from (moves the cursor on)
        const TileRef mine = next;
        const long long nc = c + stride;
        if (nc < a.n_chunks) next = locate(nc);
        // (No L2 prefetch of the next chunk's tiles: on a single launch it gains 0.5 %, but in a step that runs at the
        // board's power limit the extra L2 requests cost 1.4 %.)

        // Three passes through one copy of the transform core: 0 = DCT-II down column t of B = beta*m + g,
        // 1 = DCT-II along row t (followed by the selection and the sparse row stage of the inverse),
        // 2 = DCT-III down column t of the row-stage tile (followed by the residual).
#pragma unroll 1
        for (int ph = 0; ph < (QDOM ? 2 : 3); ++ph) {
            float w[S], y[S];
            if (ph < 2) {
                float x[S];
                if (ph == 0) {
                    if constexpr (QDOM) {
                        // row t of the stored coefficients (column t of the transposed tile) is parked for pass 1;
                        // the forward transform runs on the gradient alone
                        float mq[S];
#pragma unroll
                        for (int i = 0; i < S; ++i) mq[i] = Ms[i * S + t];
                        tmem_st64(taddr, mq);
#pragma unroll
                        for (int i = 0; i < S; ++i) x[i] = to_f32(Gs[i * S + t]);
                    } else {
#pragma unroll
                        for (int i = 0; i < S; ++i) x[i] = fmaf(a.beta, Ms[i * S + t], to_f32(Gs[i * S + t]));
                        // B = beta*m + g, parked for the residual; column k of the tensor-memory lane takes element
                        // pair_order(k), so that the registers of the store are those of the cascade's pairs
                        float xp[S];
                        fdct::static_for<0, S>([&](auto i) { xp[decltype(i)::value] = x[fdct::pair_order(decltype(i)::value)]; });
                        tmem_st64(taddr, xp);
                    }
                    // every thread has consumed its column of the staged tiles (X aliases them)
                    if (!sb.sync_and(arrived)) {
                        if (t == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
                        mbar_wait_bounded(bar, phase ^ 1u);  // give copies in flight one more bounded chance to land
                        dead = true;
                        break;
                    }
                } else {
                    const float4 *row = reinterpret_cast<const float4 *>(X + t * XS);
#pragma unroll
                    for (int v4 = 0; v4 < S / 4; ++v4) {  // (pass 0 stored the rows in pair order)
                        const float4 f = row[v4];
                        x[4 * v4 + 0] = f.x;
                        x[4 * v4 + 1] = f.y;
                        x[4 * v4 + 3] = f.z;
                        x[4 * v4 + 2] = f.w;
                    }
                }
                fdct::dct2_pre_paired<S>(x, w);
            } else {
                // column t of the row-stage tile was written by this thread only: no barrier before reading it
                fdct::static_for<0, S>([&](auto i) {
                    constexpr int p = decltype(i)::value;
                    w[p] = X[fdct::core_index<S>(p) * XS + t];
                });
            }

            fdct::dct_core_ortho_paired<S>(w, y);

            if (ph == 0) {
                // transpose through shared memory; inside a row the elements sit in pair order, so that the 128-bit
                // row reads of pass 1 deliver the cascade's pairs as they are
                float *Xc = X + fdct::pair_order(t);
                fdct::static_for<0, S>([&](auto i) {
                    constexpr int p = decltype(i)::value;
                    Xc[fdct::core_index<S>(p) * XS] = y[p];
                });
                sb.sync();
            } else if (ph == 2) {
                // m <- B - alpha * IDCT(kept): column t of the new momentum goes into a dense tile (the m staging
                // area; the row-stage tile it overlaps is dead for every thread only after the barrier below, so the
                // column is formed in registers first), which one TMA store writes out; the next chunk's tiles are
                // requested as soon as the store has read the tile.
                fdct::F2 rp[S / 2];  // pair p: rows (2p, 2p+1), swapped for odd p
                fdct::dct3_post_pairs<S>(y, rp);
                tmem_wait_st();  // the store of B (pass 0) has long completed
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float b[32];  // columns 32h .. 32h+31 of the lane: B in pair order, i.e. the pairs' own order
                    tmem_ld32(taddr + 32 * h, b);
#pragma unroll
                    for (int q = 0; q < 16; ++q) rp[16 * h + q] = fdct::f2_sub(fdct::f2_make(b[2 * q], b[2 * q + 1]), rp[16 * h + q]);
                }
                sb.sync();  // every thread has read its column of the row-stage tile
                fdct::static_for<0, S / 2>([&](auto i) {
                    constexpr int p = decltype(i)::value;
                    Ms[(2 * p + (p & 1)) * S + t] = fdct::f2_lo(rp[p]);
                    Ms[(2 * p + 1 - (p & 1)) * S + t] = fdct::f2_hi(rp[p]);
                });
                fence_proxy_async();
                sb.sync();
                {
                    // the store of this chunk, then -- once it has read the tile -- the loads of the next chunk
                    if (t == 0) {
                        tma_store_2d(mine.tm_m, mine.x, mine.y, smem_u32(Ms));
                        tma_store_commit();
                        tma_store_wait_read();
                        if (nc < a.n_chunks) issue_loads(next);
                    }
                }
            } else {
                // ---- coefficients of row t: q[v] = Q[t][v] ------------------------------------------
                float q[S];
                fdct::static_for<0, S>([&](auto i) {
                    constexpr int p = decltype(i)::value;
                    q[fdct::core_index<S>(p)] = y[p];
                });
                if constexpr (QDOM) {
                    // Q = beta * Qm + DCT(g); the stored row comes back from tensor memory
                    tmem_wait_st();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float mq[32];
                        tmem_ld32(taddr + 32 * h, mq);
#pragma unroll
                        for (int j = 0; j < 32; ++j) q[32 * h + j] = fmaf(a.beta, mq[j], q[32 * h + j]);
                    }
                    select_chunk<true>(sm, q, k_eff, rec, a.alpha, t, sb, slot + 1, PAD_ROW);
                    sb.sync();  // the tile holds Q - alpha * Q_kept (kept entries were patched by the record writers)
                    float4 rowv[S / 4];
                    {
                        const float4 *row = reinterpret_cast<const float4 *>(X + t * XS);
#pragma unroll
                        for (int v4 = 0; v4 < S / 4; ++v4) rowv[v4] = row[v4];
                    }
                    sb.sync();  // the dense tile below overlaps the coefficient tile
#pragma unroll
                    for (int v4 = 0; v4 < S / 4; ++v4) {
                        Ms[(4 * v4 + 0) * S + t] = rowv[v4].x;
                        Ms[(4 * v4 + 1) * S + t] = rowv[v4].y;
                        Ms[(4 * v4 + 2) * S + t] = rowv[v4].z;
                        Ms[(4 * v4 + 3) * S + t] = rowv[v4].w;
                    }
                    fence_proxy_async();
                    sb.sync();
                    if (t == 0) {
                        tma_store_2d(mine.tm_m, mine.x, mine.y, smem_u32(Ms));
                        tma_store_commit();
                        tma_store_wait_read();
                        if (nc < a.n_chunks) issue_loads(next);
                    }
                    continue;
                }
                select_chunk<false>(sm, q, k_eff, rec, a.alpha, t, sb, slot + 1, PAD_ROW);
                sb.sync();  // records complete (shared list and global payload), tile zeroed

                // ---- residual: row stage of the inverse from the k_eff records, sparse --------------
                {
                    // T[u][t] = sum over kept (u, v) of alpha * val * C[v][t]; the basis is read through L1
                    const float *Ct = a.C + t;
                    float acc = 0.f;
                    if (k_eff <= 64) {
                        // The running sum of a row is stored after every entry (the last store of a row carries the
                        // whole sum) and starts again from zero when the next entry belongs to another row: no branch in
                        // the loop.  The list is padded with zero-valued entries (entry 64 is always one) whose "row" is
                        // a scratch line outside the tile.  Entries and their cosines are fetched ahead of the
                        // dependent accumulation.
                        float *Xt = X + t;
                        int4 nx = recs4[0];
#pragma unroll 1
                        for (int r0 = 0; r0 < k_eff; r0 += ROW_AHEAD) {
                            int4 rc[ROW_AHEAD + 1];
                            float cv[ROW_AHEAD];
                            rc[0] = nx;
#pragma unroll
                            for (int j = 1; j < ROW_AHEAD + 1; ++j) rc[j] = recs4[r0 + j];
                            nx = rc[ROW_AHEAD];
#pragma unroll
                            for (int j = 0; j < ROW_AHEAD; ++j) cv[j] = __ldg(a.C + (unsigned)(rc[j].y + t));
#pragma unroll
                            for (int j = 0; j < ROW_AHEAD; ++j) {
                                acc = fmaf(__int_as_float(rc[j].z), cv[j], acc);
                                Xt[rc[j].x] = acc;
                                acc = (rc[j].x != rc[j + 1].x) ? 0.f : acc;
                            }
                        }
                    } else {
                        // k > 64: up to 256 kept records come from a compact shared list, more from the payload
                        // itself; four cosines are fetched ahead
                        const bool listed = k_eff <= 256;
                        int cur_u = -1;
#pragma unroll 1
                        for (int r0 = 0; r0 < k_eff; r0 += 4) {
                            int u[4];
                            float z[4], cv[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                u[j] = -1;
                                z[j] = 0.f;
                                int v = 0;
                                if (r0 + j < k_eff) {
                                    if (listed) {
                                        const uint2 e = sm.rbig[r0 + j];
                                        u[j] = (int)(e.x >> 16) * XS;
                                        v = (int)(e.x & 0xffffu);
                                        z[j] = __uint_as_float(e.y);
                                    } else {
                                        const DemoRecord rc = rec[r0 + j];
                                        u[j] = (rc.idx >> LOG2S) * XS;
                                        v = rc.idx & (S - 1);
                                        z[j] = a.alpha * rc.val;
                                    }
                                }
                                cv[j] = __ldg(Ct + v * S);
                            }
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (u[j] >= 0) {
                                    if (u[j] != cur_u) {
                                        if (cur_u >= 0) X[cur_u + t] = acc;
                                        acc = 0.f;
                                        cur_u = u[j];
                                    }
                                    acc = fmaf(z[j], cv[j], acc);
                                }
                            }
                        }
                        if (cur_u >= 0) X[cur_u + t] = acc;
                    }
                }
            }
        }
        if (dead) break;
    }
    // tear-down: every slot of the CTA is done with its tensor-memory columns
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (hw_warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
}

template <typename GT, int THREADS, bool QDOM>
cudaError_t launch64(const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    constexpr int NCH = THREADS / S;
    auto kernel = compress64_kernel<GT, THREADS, QDOM>;
    const size_t smem = slot_bytes<GT>() * NCH + 16;
    if (a.n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    // CTAs per SM: registers (launch bounds: 512 threads per SM), shared memory (227 KB, 1 KB reserved per CTA)
    // and tensor memory (512 columns, 64 per four warps).  The occupancy calculator is not asked: it does not
    // know about tensor memory and was seen to answer 1 for this kernel.
    int per_sm = 512 / THREADS;
    const int smem_limit = (int)((227u * 1024u) / (smem + 1024u));
    const int tmem_limit = 512 / (((THREADS + 127) / 128) * TMEM_COLS_PER_GROUP);
    if (per_sm > smem_limit) per_sm = smem_limit;
    if (per_sm > tmem_limit) per_sm = tmem_limit;
    if (per_sm < 1) per_sm = 1;
    const long long groups = (a.n_chunks + NCH - 1) / NCH;
    long long grid = (long long)sm_count * per_sm;
    if (grid > groups) grid = groups;
    kernel<<<(unsigned)grid, THREADS, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace

// Needs the TMA tensor maps of both tensors.
cudaError_t demo_launch_compress_fast64(const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    if (a.tmap_m == nullptr || a.tmap_g == nullptr) return cudaErrorNotSupported;
#ifndef DEMO_T64
#define DEMO_T64 64
#endif
    if (a.momentum_dct)
        return a.grad_bf16 ? launch64<__nv_bfloat16, DEMO_T64, true>(a, sm_count, stream)
                           : launch64<float, DEMO_T64, true>(a, sm_count, stream);
    return a.grad_bf16 ? launch64<__nv_bfloat16, DEMO_T64, false>(a, sm_count, stream)
                       : launch64<float, DEMO_T64, false>(a, sm_count, stream);
}
