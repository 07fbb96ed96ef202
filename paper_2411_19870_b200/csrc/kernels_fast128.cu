// Fast kernels for 2-D tensors with chunk size 128: one 256-thread CTA per 128 x 128 chunk.
//
// A 128-point transform does not fit one thread's registers, so it is split by the first stage of the
// same factorisation the 64-point code uses (fast_dct.cuh):
//     DCT-II_128:  u[n] = x[n] + x[127-n],  v[n] = x[n] - x[127-n]   (n < 64)
//                  X[2p] = DCT-II_64(u)[p],  X[2p+1] = DCT-IV_64(v)[p]
// Thread (h, j) = (threadIdx.x / 128, threadIdx.x % 128) owns line j (a column in the first pass, a row
// in the second) and computes its even (h = 0) or odd (h = 1) outputs; h is warp-uniform, so the two
// transform bodies never diverge inside a warp.  The inverse runs the transposed graph:
//     e = DCT-III_64(X[even]),  o = DCT-IV_64(X[odd]),  x[n] = e[n] + o[n],  x[127-n] = e[n] - o[n]
// with e and o exchanged between the two threads of a line through shared memory.
//
// compress: TMA-staged m and g tiles -> B = beta*m + g (each thread parks the half column it will write back in
// tensor memory) -> column pass -> row pass -> coefficients in shared memory -> exact top-k (bound from the 256
// half-row maxima, candidate list, exact ranking; radix select for degenerate chunks) -> records; sparse row
// stage of the inverse from the records, fast column stage, residual m <- B - alpha * IDCT(kept) against the
// parked B, one TMA store of the new momentum tile.  decode: scatter-add of the W payloads in worker order,
// two inverse passes, sign, update; the x tile is staged into the (then dead) coefficient tile.
// Tiles need the TMA tensor maps; without them the host uses the generic kernels for s = 128.
#include <cuda_bf16.h>

#include "demo_internal.h"
#include "fast_common.cuh"
#include "fast_dct.cuh"

namespace {

using namespace fastk;

constexpr int S = 128, H = 64, XS = S + 4, M = S * S, THREADS = 256;
// The decode tile is only ever accessed element-wise: an odd row stride keeps a warp whose lanes walk 32
// different rows (the row pass) on 32 different banks; S + 4 (compress: 128-bit row accesses) gives 4-way
// conflicts there.
constexpr int XSD = S + 1;
constexpr int RECS128 = 128 + 40;     // row-stage list: up to 128 kept records + padding for the look-ahead
constexpr int ROW_AHEAD128 = 8;       // entries of the row-stage list fetched ahead of the accumulation
constexpr int TMEM_COLS128 = 128;     // tensor-memory columns of a compress CTA (two CTAs per SM)
constexpr int CAP128 = 256;           // candidate capacity of the fast top-k (one per thread)
constexpr int CAP128P = CAP128 + 4;   // padded for 128-bit key loads
using SC = fdct::ScaleOrtho<S>;

__device__ __forceinline__ unsigned block_exclusive_scan(unsigned v, unsigned *warp_tot /*[8]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned inc = warp_inclusive_scan(v, lane);
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    unsigned base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    __syncthreads();
    return base + inc - v;
}

// Forward half-transform of one line: in[n] = x[n] (+/-) x[127-n] already formed; out[p] is
// coefficient 2p (h = 0) or 2p+1 (h = 1) of the orthonormal 128-point DCT-II.
__device__ __forceinline__ void forward_half(int h, float (&in)[H], float (&out)[H])
{
    if (h == 0) {
        fdct::dct2_packed<H, SC>(in, out);
        out[0] *= fdct::dc_scale<S>();
    } else {
        fdct::dct4_paired<H, SC>(in, out);
    }
}
// Inverse half-transform: in[p] = coefficient 2p (h = 0) or 2p+1 (h = 1); out = e (h = 0) or o (h = 1).
__device__ __forceinline__ void inverse_half(int h, float (&in)[H], float (&out)[H])
{
    if (h == 0) {
        in[0] *= fdct::dc_scale<S>();
        fdct::dct3_packed<H, SC>(in, out);
    } else {
        fdct::dct4_paired<H, SC>(in, out);
    }
}

template <typename GT>
constexpr size_t compress128_tile_bytes()
{
    return (size_t)M * (sizeof(float) + sizeof(GT)) > (size_t)S * XS * 4 ? (size_t)M * (sizeof(float) + sizeof(GT))
                                                                         : (size_t)S * XS * 4;
}
template <typename GT>
constexpr size_t compress128_smem()
{
    return compress128_tile_bytes<GT>() + (256 + 8 + 4) * 4 + RECS128 * 16 + 3 * CAP128P * 4 + 16 + 16;
}

template <typename GT>
__global__ void __launch_bounds__(THREADS, 2) compress_fast128_kernel(DemoCompressArgs a)
{
    constexpr unsigned TILE_BYTES = M * sizeof(float) + M * sizeof(GT);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *Ms = reinterpret_cast<float *>(smem_raw);  // [128*128] m tile
    GT *Gs = reinterpret_cast<GT *>(Ms + M);          // [128*128] g tile
    float *X = Ms;                                    // [128*132] transpose / coefficients / row stage (aliases the tiles)
    unsigned *hist = reinterpret_cast<unsigned *>(smem_raw + compress128_tile_bytes<GT>());  // [256]
    unsigned *warp_tot = hist + 256;                                                         // [8]
    unsigned *s_state = warp_tot + 8;                                                        // [4]
    int4 *recs4 = reinterpret_cast<int4 *>(s_state + 4);                                     // [RECS128]
    unsigned *cand_key = reinterpret_cast<unsigned *>(recs4 + RECS128);                      // [CAP128P]
    float *cand_val = reinterpret_cast<float *>(cand_key + CAP128P);                         // [CAP128P]
    int *cand_idx = reinterpret_cast<int *>(cand_val + CAP128P);                             // [CAP128P]
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(cand_idx + CAP128P);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_mem + 2);

    const int tid = threadIdx.x, h = tid >> 7, j = tid & 127;
    const uint32_t bar = smem_u32(bar_mem);
    if (tid == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();
    }
    // Tensor memory as storage: thread (h, j) parks its 64 elements of column j of B = beta*m + g (rows 0..63 for
    // h = 0, rows 127..64 for h = 1) in lane j, columns 64h .. 64h+63, between the forward pass and the residual.
    const uint32_t tmem_base = tmem_alloc_cta(tmem_slot, TMEM_COLS128);
    fence_proxy_async();
    const uint32_t taddr = tmem_base + ((uint32_t)(j & ~31) << 16) + (uint32_t)(h * H);

    EntryCursor cur;
    unsigned phase = 0;
    const char *acquired = nullptr;

    auto issue_tiles = [&](const DemoTensorEntry &te, long long c) {
        const unsigned lc = (unsigned)(c - te.chunk_begin);
        const unsigned k0 = lc / (unsigned)te.c1, k1 = lc - k0 * (unsigned)te.c1;
        if (tid == 0) {
            const char *tm_m = static_cast<const char *>(a.tmap_m) + (size_t)te.tensor * TMAP_BYTES;
            const char *tm_g = static_cast<const char *>(a.tmap_g) + (size_t)te.tensor * TMAP_BYTES;
            if (tm_m != acquired) {  // a tensor map this thread has not used yet: acquire it for the tensor-map proxy
                acquired = tm_m;
                tmap_acquire(tm_m);
                tmap_acquire(tm_g);
            }
            mbar_expect_tx(bar, TILE_BYTES);
            tma_load_2d(smem_u32(Ms), tm_m, k1 * S, k0 * S, bar);
            tma_load_2d(smem_u32(Gs), tm_g, k1 * S, k0 * S, bar);
        }
    };

    long long c = blockIdx.x;
    if (c < a.n_chunks) {
        cur.seek(a.entries, a.n_entries, c);
        issue_tiles(cur.te, c);
    }
    for (; c < a.n_chunks; c += gridDim.x) {
        const DemoTensorEntry te = cur.te;  // the cursor points at chunk c
        const unsigned lc = (unsigned)(c - te.chunk_begin);
        const unsigned k0 = lc / (unsigned)te.c1, k1 = lc - k0 * (unsigned)te.c1;
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ m = a.m_ptrs[te.tensor];
        const int k_eff = te.k_eff;
        DemoRecord *rec = a.payload + te.rec_begin + (long long)lc * k_eff;

        const bool arrived = mbar_wait_bounded(bar, phase);
        phase ^= 1u;
        if (!__syncthreads_and(arrived)) {
            if (tid == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);  // give copies in flight one more bounded chance to land
            break;
        }

        // ---- two forward passes through one rolled copy of the half-transforms ---------------------
        float in[H], out[H];
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            if (pass == 0) {
                // column j of B = beta*m + g, folded: in[n] = B[n][j] +/- B[127-n][j]; the half of the column that
                // this thread will write back is parked in tensor memory (two stores of 32 columns)
                const float sg = h ? -1.f : 1.f;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    float park[32];
#pragma unroll
                    for (int q = 0; q < 32; ++q) {
                        const int n = 32 * half + q;
                        const float lo = fmaf(a.beta, Ms[n * S + j], to_f32(Gs[n * S + j]));
                        const float hi = fmaf(a.beta, Ms[(S - 1 - n) * S + j], to_f32(Gs[(S - 1 - n) * S + j]));
                        in[n] = fmaf(sg, hi, lo);
                        park[q] = h ? hi : lo;
                    }
                    tmem_st32(taddr + 32 * half, park);
                }
                __syncthreads();  // the staged tiles are consumed (X aliases them)
            } else {
                // row j of the column-transformed tile, folded
                const float4 *row = reinterpret_cast<const float4 *>(X + j * XS);
#pragma unroll
                for (int n4 = 0; n4 < H / 4; ++n4) {
                    const float4 lo = row[n4];
                    const float4 hi = row[S / 4 - 1 - n4];  // elements 127-4n4-3 .. 127-4n4
                    in[4 * n4 + 0] = h ? lo.x - hi.w : lo.x + hi.w;
                    in[4 * n4 + 1] = h ? lo.y - hi.z : lo.y + hi.z;
                    in[4 * n4 + 2] = h ? lo.z - hi.y : lo.z + hi.y;
                    in[4 * n4 + 3] = h ? lo.w - hi.x : lo.w + hi.x;
                }
                __syncthreads();  // every thread has read its row before the coefficients overwrite the tile
            }
            forward_half(h, in, out);
            if (pass == 0) {
#pragma unroll
                for (int p = 0; p < H; ++p) X[(2 * p + h) * XS + j] = out[p];  // Y[u][j]
            } else {
                // Q[j][2p + h]: a row keeps its even coefficients in its first half and its odd ones in the second
                // (position 64h + p), so that each thread stores its 64 outputs with 128-bit stores; element-wise
                // stores along a row, with a warp's lanes on 32 different rows, would run into 4-way bank conflicts
                float4 *dst = reinterpret_cast<float4 *>(X + j * XS + H * h);
#pragma unroll
                for (int p4 = 0; p4 < H / 4; ++p4) dst[p4] = make_float4(out[4 * p4], out[4 * p4 + 1], out[4 * p4 + 2], out[4 * p4 + 3]);
            }
            __syncthreads();
        }

        // ---- exact top-k ---------------------------------------------------------------------------
        // thread tid scans one half of row tid/2 as the row pass stored it: the even coefficients (tid even) or the
        // odd ones (tid odd); element e of its half is coefficient 2e + (tid & 1), flat index 128*(tid/2) + 2e + (tid&1).
        // Fast path (k_eff <= 256): the k_eff-th largest of the 256 per-thread maxima is a lower bound L of
        // the k_eff-th largest coefficient (256 groups: the bound is tight, a few dozen candidates); the
        // candidates are listed in index order and ranked exactly, ties to the lowest index.  Everything
        // compares integer magnitude keys, so NaN and Inf are ordered like any other bit pattern.  More
        // than CAP128 candidates (tied or degenerate chunks) or k_eff > 256: radix select below.
        // the row-stage list is padded with zero-valued entries whose "row" is a scratch line behind the tile
        // (ordered before the record writes by the barriers below)
        if (tid < RECS128) recs4[tid] = make_int4(S * XS, 0, 0, 0);
        bool use_radix = k_eff > 256;
        if (!use_radix) {
            const float4 *mine4 = reinterpret_cast<const float4 *>(X + (tid >> 1) * XS + 64 * (tid & 1));
            const int lane = tid & 31, warp = tid >> 5;
            // the two halves of a row sit 256 bytes apart (same banks): the odd one starts 4 pieces later
            const int rot = 4 * (tid & 1);
            // the 64 values stay in registers for the candidate mask (group i4 holds piece (i4 + rot) mod 16)
            float v[64];
            float tm = 0.f;
#pragma unroll
            for (int i4 = 0; i4 < 16; ++i4) {
                const float4 f = mine4[(i4 + rot) & 15];
                v[4 * i4 + 0] = f.x;
                v[4 * i4 + 1] = f.y;
                v[4 * i4 + 2] = f.z;
                v[4 * i4 + 3] = f.w;
                tm = max3f(tm, fabsf(f.x), fabsf(f.y));
                tm = max3f(tm, fabsf(f.z), fabsf(f.w));
            }
            const unsigned tkey = __float_as_uint(tm);
            hist[tid] = tkey;
            __syncthreads();
            if (warp == 0) {
                unsigned k8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) k8[i] = hist[lane + 32 * i];
                unsigned lo = k8[0], hi = k8[0];
#pragma unroll
                for (int i = 1; i < 8; ++i) {
                    lo = min(lo, k8[i]);
                    hi = max(hi, k8[i]);
                }
                lo = __reduce_min_sync(0xffffffffu, lo);
                hi = __reduce_max_sync(0xffffffffu, hi);
                const int b0 = 31 - __clz((lo ^ hi) | 0x8000u);  // >= 15
                unsigned prefix = lo & ~((2u << b0) - 1u);
#pragma unroll 1
                for (int b = b0; b >= 15; --b) {
                    const unsigned cand = prefix | (1u << b);
                    unsigned cnt = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) cnt += __popc(__ballot_sync(0xffffffffu, k8[i] >= cand));
                    prefix = (cnt >= (unsigned)k_eff) ? cand : prefix;
                }
                if (lane == 0) {
                    s_state[2] = prefix;
                    s_state[3] = hi;  // largest magnitude key of the chunk (read before the scan below reuses the word)
                }
            }
            __syncthreads();
            const unsigned lmin = s_state[2];
            // every coefficient zero (a tile that no gradient has touched yet): no selection needed, the tie
            // rule gives the records 0 .. k_eff-1 with value 0
            const bool zero_chunk = s_state[3] == 0u;
            if (zero_chunk) {
                if (tid < k_eff) {
                    DemoRecord r;
                    r.idx = tid;
                    r.val = 0.f;
                    rec[tid] = r;
                    if (k_eff <= 128) recs4[tid] = make_int4((tid >> 7) * XS, (tid & 127) * S, 0, 0);
                }
            } else {
            // candidates of this thread as a bit mask over its 64 values: |q| >= L  <=>  |q| > Lm (the float just
            // below L); the sign bit of Lm - |q| is funnel-shifted into the mask (independent chains of 16), which is
            // then turned from register order into index order
            unsigned long long mask;
            {
                const float Lm = (lmin > 0u) ? __uint_as_float(lmin - 1u) : -1.f;
                unsigned mc[4];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    unsigned mm = 0u;
#pragma unroll
                    for (int q = 15; q >= 0; --q) mm = __funnelshift_l(__float_as_uint(Lm - fabsf(v[16 * ch + q])), mm, 1);
                    mc[ch] = mm;
                }
                const unsigned long long mreg =
                    ((unsigned long long)(mc[2] | (mc[3] << 16)) << 32) | (unsigned long long)(mc[0] | (mc[1] << 16));
                mask = (tid & 1) ? ((mreg << 16) | (mreg >> 48)) : mreg;
            }
            const unsigned cnt = (unsigned)__popcll(mask);
            const unsigned o = block_exclusive_scan(cnt, warp_tot);
            if (tid == THREADS - 1) s_state[3] = o + cnt;
            __syncthreads();
            const unsigned n_cand = s_state[3];
            use_radix = n_cand > (unsigned)CAP128 || n_cand < (unsigned)k_eff;
            if (!use_radix) {
                // The list is in index order: inside a row the candidates of the even-coefficient thread (lane 2r)
                // and of the odd-coefficient thread (lane 2r+1) interleave, so a candidate's place is the row's base
                // plus the candidates of both threads with a smaller coefficient index.
                const unsigned plo = __shfl_xor_sync(0xffffffffu, (unsigned)mask, 1);
                const unsigned phi = __shfl_xor_sync(0xffffffffu, (unsigned)(mask >> 32), 1);
                const unsigned long long pmask = ((unsigned long long)phi << 32) | plo;
                const int odd = tid & 1;
                const unsigned row_base = odd ? o - (unsigned)__popcll(pmask) : o;
                const float *mine = reinterpret_cast<const float *>(mine4);
                unsigned long long left = mask;
                while (left) {
                    const int e = __ffsll((long long)left) - 1;
                    left &= left - 1ull;
                    const unsigned long long below = (1ull << e) - 1ull;
                    // partner coefficients before 2e + odd: 2e' + (1 - odd) with e' < e (even thread) or e' <= e (odd thread)
                    const unsigned long long pbelow = odd ? ((below << 1) | 1ull) : below;
                    const unsigned at = row_base + (unsigned)__popcll(mask & below) + (unsigned)__popcll(pmask & pbelow);
                    const float val = mine[e];
                    cand_key[at] = mag_key(val);
                    cand_val[at] = val;
                    cand_idx[at] = S * (tid >> 1) + 2 * e + odd;
                }
                __syncthreads();
                // the first warp picks the k_eff largest candidates (list order = index order) and writes the records
                if (warp == 0) {
                    auto emit = [&](unsigned pos, unsigned li) {
                        DemoRecord r;
                        r.idx = cand_idx[li];
                        r.val = cand_val[li];
                        rec[pos] = r;
                        if (k_eff <= 128)
                            recs4[pos] = make_int4((r.idx >> 7) * XS, (r.idx & 127) * S, __float_as_int(a.alpha * r.val), 0);
                    };
                    auto where = [](unsigned i) { return i; };
                    if (n_cand <= 64u)
                        warp_ballot_select<2>(cand_key, n_cand, lmin, k_eff, lane, where, emit);
                    else
                        warp_ballot_select<8>(cand_key, n_cand, lmin, k_eff, lane, where, emit);
                }
            }
            }  // !zero_chunk
        }
        // ---- radix select on the magnitude bits, then index-ordered compaction -----------------------
        if (use_radix) {
            unsigned thr, need_eq;
            if (tid == 0) {
                s_state[0] = 0u;
                s_state[1] = (unsigned)k_eff;
            }
            // this path works on rows in natural order: every thread turns its half row back (coefficient 2e + (tid&1)
            // from position 64*(tid&1) + e to position 2e + (tid&1)); then thread tid scans the half row
            // [tid/2][64*(tid&1) .. +64): flat indices 64*tid .. 64*tid+63
            {
                float *rowp = X + (tid >> 1) * XS;
                float tmp[64];
#pragma unroll
                for (int i4 = 0; i4 < 16; ++i4) {
                    const float4 f = reinterpret_cast<const float4 *>(rowp + 64 * (tid & 1))[i4];
                    tmp[4 * i4 + 0] = f.x;
                    tmp[4 * i4 + 1] = f.y;
                    tmp[4 * i4 + 2] = f.z;
                    tmp[4 * i4 + 3] = f.w;
                }
                __syncthreads();
#pragma unroll
                for (int e = 0; e < 64; ++e) rowp[2 * e + (tid & 1)] = tmp[e];
                __syncthreads();
            }
            const float *mine = X + (tid >> 1) * XS + 64 * (tid & 1);
#pragma unroll 1
            for (int pass = 0; pass < 4; ++pass) {
                const int shift = 24 - 8 * pass;
                const unsigned mask = (pass == 0) ? 0u : (0xffffffffu << (shift + 8));
                hist[tid] = 0u;
                __syncthreads();
                const unsigned prefix = s_state[0];
#pragma unroll 4
                for (int e = 0; e < 64; ++e) {
                    const unsigned key = mag_key(mine[e]);
                    if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
                }
                __syncthreads();
                if (tid < 32) {
                    const unsigned rem = s_state[1];
                    unsigned local = 0;
#pragma unroll
                    for (int b = 0; b < 8; ++b) local += hist[255 - 8 * tid - b];
                    const unsigned inc = warp_inclusive_scan(local, tid);
                    const unsigned before = inc - local;
                    if (before < rem && rem <= inc) {
                        unsigned cum = before;
                        int b = 255 - 8 * tid;
                        for (int q = 0; q < 8; ++q, --b) {
                            const unsigned hh = hist[b];
                            if (cum + hh >= rem) break;
                            cum += hh;
                        }
                        s_state[1] = rem - cum;
                        s_state[0] = prefix | ((unsigned)b << shift);
                    }
                }
                __syncthreads();
            }
            thr = s_state[0];
            need_eq = s_state[1];
            unsigned gt = 0, eq = 0;
#pragma unroll 4
            for (int e = 0; e < 64; ++e) {
                const unsigned key = mag_key(mine[e]);
                gt += key > thr;
                eq += key == thr;
            }
            const unsigned before = block_exclusive_scan(gt | (eq << 16), warp_tot);
            unsigned gb = before & 0xffffu, eb = before >> 16;
#pragma unroll 1
            for (int e = 0; e < 64; ++e) {
                const float val = mine[e];
                const unsigned key = mag_key(val);
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
                    const int idx = 64 * tid + e;
                    DemoRecord r;
                    r.idx = idx;
                    r.val = val;
                    rec[pos] = r;
                    if (k_eff <= 128)
                        recs4[pos] = make_int4((idx >> 7) * XS, (idx & 127) * S, __float_as_int(a.alpha * val), 0);
                }
            }
        }
        __syncthreads();  // records complete; the coefficient tile is dead

        // ---- residual: sparse row stage T[u][j] = sum over kept (u, v) of val * C[v][j] ------------
        for (int i = tid; i < S * XS / 4; i += THREADS) reinterpret_cast<float4 *>(X)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncthreads();
        if (h == 0 && k_eff <= 128) {
            // The running sum of a row is stored after every entry (the last store of a row carries the whole sum)
            // and starts again from zero when the next entry belongs to another row: no branch in the loop.
            // The cosines of a whole batch of entries are requested before the dependent accumulation starts: the
            // 64 KB basis does not stay in what the two CTAs' shared memory leaves of the L1, so most of these
            // loads go to L2 and a batch should pay that latency once.
            float *Xj = X + j;
            float acc = 0.f;
            auto row_stage = [&](auto batch_tag) {
                constexpr int BATCH = decltype(batch_tag)::value;
#pragma unroll 1
                for (int r0 = 0; r0 < k_eff; r0 += BATCH) {
                    float cv[BATCH];
#pragma unroll
                    for (int q = 0; q < BATCH; ++q) cv[q] = __ldg(a.C + (unsigned)(recs4[r0 + q].y + j));
                    int4 nx = recs4[r0];
#pragma unroll
                    for (int q = 0; q < BATCH; ++q) {
                        const int4 rc = nx;
                        nx = recs4[r0 + q + 1];
                        acc = fmaf(__int_as_float(rc.z), cv[q], acc);
                        Xj[rc.x] = acc;
                        acc = (rc.x != nx.x) ? 0.f : acc;
                    }
                }
            };
            if (k_eff <= ROW_AHEAD128)
                row_stage(std::integral_constant<int, ROW_AHEAD128>{});
            else
                row_stage(std::integral_constant<int, 4 * ROW_AHEAD128>{});
        } else if (h == 0) {
            // k > 128: the records come from the payload itself
            const float *Cj = a.C + j;
            float acc = 0.f;
            int cur_u = -1;
            for (int r = 0; r < k_eff; ++r) {
                const DemoRecord rc = rec[r];
                const int uo = (rc.idx >> 7) * XS;
                if (uo != cur_u) {
                    if (cur_u >= 0) X[cur_u + j] = acc;
                    acc = 0.f;
                    cur_u = uo;
                }
                acc = fmaf(a.alpha * rc.val, __ldg(Cj + (rc.idx & 127) * S), acc);
            }
            if (cur_u >= 0) X[cur_u + j] = acc;
        }
        __syncthreads();

        // ---- column stage of the inverse (split), second fetch of the tiles, residual --------------
#pragma unroll
        for (int p = 0; p < H; ++p) in[p] = X[(2 * p + h) * XS + j];
        fence_proxy_async();
        __syncthreads();  // T is in registers: the tile area is free
        inverse_half(h, in, out);
        // exchange e and o through the tile area
        float *Ex = X;  // [2][64][128]
#pragma unroll
        for (int n = 0; n < H; ++n) Ex[(h * H + n) * S + j] = out[n];
        __syncthreads();
#pragma unroll
        for (int n = 0; n < H; ++n) {
            const float other = Ex[((h ^ 1) * H + n) * S + j];
            out[n] = h ? other - out[n] : out[n] + other;  // h=0: x[n] = e+o;  h=1: x[127-n] = e-o
        }
        __syncthreads();  // the exchange area is read: the new momentum tile takes its place
        // m <- B - alpha * IDCT(kept): B comes back from tensor memory; the dense tile goes out in one TMA store
        tmem_wait_st();
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float b[32];
            tmem_ld32(taddr + 32 * half, b);
            if (h) {
#pragma unroll
                for (int q = 0; q < 32; ++q) Ms[(S - 1 - (32 * half + q)) * S + j] = b[q] - out[32 * half + q];
            } else {
#pragma unroll
                for (int q = 0; q < 32; ++q) Ms[(32 * half + q) * S + j] = b[q] - out[32 * half + q];
            }
        }
        fence_proxy_async();
        __syncthreads();
        const long long nc = c + gridDim.x;
        if (nc < a.n_chunks) cur.seek(a.entries, a.n_entries, nc);
        if (tid == 0) {
            tma_store_2d(static_cast<const char *>(a.tmap_m) + (size_t)te.tensor * TMAP_BYTES, (int)(k1 * S), (int)(k0 * S),
                         smem_u32(Ms));
            tma_store_commit();
            tma_store_wait_read();  // the store has read the tile: the next chunk's tiles may land
        }
        if (nc < a.n_chunks) issue_tiles(cur.te, nc);
    }
    tmem_free_cta(tmem_base, TMEM_COLS128);
}

constexpr size_t decode128_smem(bool counts) { return (size_t)S * XSD * 4 + 16 + (counts ? (size_t)M * 2 : 0); }

// SIGNS: the parameter-server form -- sign(R) goes out as int8, the parameters are not touched.
template <bool SIGNS>
__global__ void __launch_bounds__(THREADS, 2) decode_fast128_kernel(DemoDecodeArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *St = reinterpret_cast<float *>(smem_raw);  // [128*132] aggregate / intermediate; later the x tile [128*128]
    float *Xt = St;
    unsigned long long *bar_mem = reinterpret_cast<unsigned long long *>(St + S * XSD);
    unsigned short *Cn = reinterpret_cast<unsigned short *>(bar_mem + 2);  // [M] senders per coordinate (agg == 2)

    const int tid = threadIdx.x, h = tid >> 7, j = tid & 127;
    const uint32_t bar = smem_u32(bar_mem);
    if (tid == 0) {
        mbar_init(bar, 1);
        fence_proxy_async();
    }
    __syncthreads();
    fence_proxy_async();

    EntryCursor cur;
    unsigned phase = 0;
    const unsigned lr_bits = __float_as_uint(a.lr);
    const float decay = 1.f - a.lr * a.wd;
    const float neg_lr_scale = -a.lr * a.agg_scale;
    const bool counts = a.agg == 2;
    const char *acquired = nullptr;

    for (long long c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
        cur.seek(a.entries, a.n_entries, c);
        const DemoTensorEntry te = cur.te;
        const unsigned lc = (unsigned)(c - te.chunk_begin);
        const unsigned k0 = lc / (unsigned)te.c1, k1 = lc - k0 * (unsigned)te.c1;
        const size_t base = (size_t)k0 * S * (size_t)te.n1 + (size_t)k1 * S;
        float *__restrict__ x = a.x_ptrs[te.tensor];
        const int k_eff = te.k_eff;
        const long long rec_off = te.rec_begin + (long long)lc * k_eff;
        const char *tm_x = static_cast<const char *>(a.tmap_x) + (size_t)te.tensor * TMAP_BYTES;
        if (!SIGNS && tid == 0) {
            if (tm_x != acquired) {  // first use of this tensor's map by this thread
                acquired = tm_x;
                tmap_acquire(tm_x);
            }
            tma_prefetch_2d(tm_x, k1 * S, k0 * S);
        }

        for (int i = tid; i < S * XSD / 4; i += THREADS) reinterpret_cast<float4 *>(St)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (counts)
            for (int i = tid; i < M; i += THREADS) Cn[i] = 0;
        __syncthreads();
        // S = sum over workers in worker order (a barrier per worker fixes the order of additions)
        for (int kb = 0; kb < k_eff; kb += THREADS) {
            const bool mine = kb + tid < k_eff;
            for (int w0 = 0; w0 < a.W; w0 += 8) {
                DemoRecord r[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (mine && w0 + q < a.W) r[q] = a.payloads[w0 + q][rec_off + kb + tid];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (w0 + q < a.W) {
                        if (mine) {
                            if ((unsigned)r[q].idx < (unsigned)M) {
                                St[(r[q].idx >> 7) * XSD + (r[q].idx & 127)] += r[q].val;
                                if (counts) Cn[r[q].idx] += 1;
                            } else {
                                atomicMax(a.status, DEMO_DEV_PAYLOAD);
                            }
                        }
                        __syncthreads();
                    }
                }
            }
        }
        if (counts) {  // Sparse Top-k Averaging: sum / number of senders, 0/0 = 0
            for (int i = tid; i < M; i += THREADS) {
                const unsigned short n = Cn[i];
                if (n > 1) St[(i >> 7) * XSD + (i & 127)] /= (float)n;
            }
            __syncthreads();
        }
        // two inverse passes (rolled): both walk "row j" of the tile with unit stride -- pass 0 leaves its result
        // transposed, so that the columns pass 1 needs are rows again and every access below has a fixed offset
        float in[H], out[H];
        bool arrived = true;
        float *ln = St + j * XSD;  // line j
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
            for (int p = 0; p < H; ++p) in[p] = ln[2 * p + h];
            fence_proxy_async();
            __syncthreads();  // every coefficient of the tile has been read
            inverse_half(h, in, out);
            // exchange e / o inside the line: e at elements 0..63, o at 64..127
#pragma unroll
            for (int n = 0; n < H; ++n) ln[h * H + n] = out[n];
            __syncthreads();
#pragma unroll
            for (int n = 0; n < H; ++n) {
                const float other = ln[(h ^ 1) * H + n];
                out[n] = h ? other - out[n] : out[n] + other;  // h=0: element n;  h=1: element 127-n
            }
            fence_proxy_async();
            __syncthreads();  // both halves of every line have read their partner's values
            if (pass == 0) {
                // element n (resp. 127-n) of row j goes to row n (127-n), column j
                if (h) {
#pragma unroll
                    for (int n = 0; n < H; ++n) St[(S - 1 - n) * XSD + j] = out[n];
                } else {
#pragma unroll
                    for (int n = 0; n < H; ++n) St[n * XSD + j] = out[n];
                }
                __syncthreads();
            } else if (!SIGNS) {
                if (tid == 0) {
                    mbar_expect_tx(bar, M * sizeof(float));
                    tma_load_2d(smem_u32(Xt), tm_x, k1 * S, k0 * S, bar);
                }
                arrived = mbar_wait_bounded(bar, phase);
                phase ^= 1u;
            }
        }
        if constexpr (SIGNS) {
            signed char *__restrict__ sg = a.sign_ptrs[te.tensor];
#pragma unroll
            for (int n = 0; n < H; ++n) {
                const int row = h ? (S - 1 - n) : n;
                sg[base + (size_t)row * te.n1 + j] = (signed char)((out[n] > 0.f) - (out[n] < 0.f));
            }
            __syncthreads();
            continue;
        }
        if (!__syncthreads_and(arrived)) {
            if (tid == 0) atomicMax(a.status, DEMO_DEV_TIMEOUT);
            mbar_wait_bounded(bar, phase ^ 1u);
            return;
        }
#pragma unroll
        for (int n = 0; n < H; ++n) {
            const int row = h ? (S - 1 - n) : n;
            const float rv = out[n];
            float stepv = __uint_as_float(lr_bits ^ (~__float_as_uint(rv) & 0x80000000u));
            stepv = (rv == 0.f) ? 0.f : stepv;
            if (a.phi) stepv = rv * neg_lr_scale;  // phi = identity
            x[base + (size_t)row * te.n1 + j] = fmaf(Xt[row * S + j], decay, stepv);
        }
        fence_proxy_async();
        __syncthreads();
    }
}

template <typename K>
cudaError_t launch128(K kernel, size_t smem, long long n_chunks, int sm_count, cudaStream_t stream, const void *args)
{
    if (n_chunks <= 0) return cudaSuccess;
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    // CTAs per SM: two by the launch bounds (registers), fewer if shared memory (227 KB, 1 KB reserved per CTA) says
    // so.  The occupancy calculator is not asked: it answers 1 for a kernel that allocates tensor memory.
    int per_sm = (int)((227u * 1024u) / (smem + 1024u));
    if (per_sm > 2) per_sm = 2;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count * per_sm;
    if (grid > n_chunks) grid = n_chunks;
    void *params[] = {const_cast<void *>(args)};
    return cudaLaunchKernel((const void *)kernel, dim3((unsigned)grid), dim3(THREADS), params, smem, stream);
}

}  // namespace

cudaError_t demo_launch_compress_fast128(const DemoCompressArgs &a, int sm_count, cudaStream_t stream)
{
    if (!a.tmap_m || !a.tmap_g) return cudaErrorNotSupported;
    if (a.grad_bf16)
        return launch128(compress_fast128_kernel<__nv_bfloat16>, compress128_smem<__nv_bfloat16>(), a.n_chunks, sm_count,
                         stream, &a);
    return launch128(compress_fast128_kernel<float>, compress128_smem<float>(), a.n_chunks, sm_count, stream, &a);
}

cudaError_t demo_launch_decode_fast128(const DemoDecodeArgs &a, int sm_count, cudaStream_t stream)
{
    if (a.sign_ptrs) return launch128(decode_fast128_kernel<true>, decode128_smem(a.agg == 2), a.n_chunks, sm_count, stream, &a);
    if (!a.tmap_x) return cudaErrorNotSupported;
    return launch128(decode_fast128_kernel<false>, decode128_smem(a.agg == 2), a.n_chunks, sm_count, stream, &a);
}
