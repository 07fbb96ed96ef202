// Register-resident fast DCT-II / DCT-III of compile-time length N (power of two), fully unrolled,
// every twiddle an immediate.  Used for the chunk DCT of the paper (Section 2.1: the projection
// matrices are the fixed orthonormal DCT basis), where it replaces the dense s x s contraction:
// about 9 flop per element and pass instead of 2s.
//
// Factorisation (all steps are butterflies or plane rotations, so rounding errors do not grow
// beyond O(log N) ulps of the data scale -- no division by small cosines, no running recurrences):
//   DCT-II_N :  u[n] = x[n] + x[N-1-n],  v[n] = x[n] - x[N-1-n]            (n < N/2)
//               X[2j] = DCT-II_{N/2}(u)[j],   X[2j+1] = DCT-IV_{N/2}(v)[j]
//   DCT-IV_N :  with th_n = (2n+1) pi / (4N), H = N/2, for n < H
//               a[n] =          v[n] cos th_n + v[N-1-n] sin th_n
//               b[n] = (-1)^n (-v[n] sin th_n + v[N-1-n] cos th_n)
//               A = DCT-II_H(a),  Bt = DCT-II_H(b)
//               V[0] = A[0],  V[2p-1] = A[p] - Bt[H-p],  V[2p] = A[p] + Bt[H-p]  (0 < p < H),
//               V[N-1] = -Bt[0]
//   DCT-III_N (transpose of DCT-II_N; DCT-IV is symmetric so it is its own transpose):
//               e = DCT-III_{N/2}(X[even]),  o = DCT-IV_{N/2}(X[odd]),
//               x[n] = e[n] + o[n],  x[N-1-n] = e[n] - o[n]
// Transforms here are un-normalised except for one scale SC applied to every output whose index
// is not 0 (folded into the rotation constants, so it is free); the caller scales the DC term.
// With SC = sqrt(2/N) and DC * sqrt(1/N) this is the orthonormal DCT-II (and its inverse).
#pragma once

#include <type_traits>

#if defined(__CUDACC__)
#define FDCT_HD __host__ __device__ __forceinline__
#else
#define FDCT_HD inline
#endif

namespace fdct {

constexpr double kPi = 3.141592653589793238462643383279502884;

constexpr double c_sqrt(double x)
{
    double r = x > 1.0 ? x : 1.0;
    for (int i = 0; i < 200; ++i) r = 0.5 * (r + x / r);
    return r;
}
// Taylor series; |x| <= pi/2 in every use below, where 16 terms reach double precision.
constexpr double c_sin(double x)
{
    double term = x, sum = x;
    for (int i = 1; i < 18; ++i) {
        term *= -x * x / ((2.0 * i) * (2.0 * i + 1.0));
        sum += term;
    }
    return sum;
}
constexpr double c_cos(double x)
{
    double term = 1.0, sum = 1.0;
    for (int i = 1; i < 18; ++i) {
        term *= -x * x / ((2.0 * i - 1.0) * (2.0 * i));
        sum += term;
    }
    return sum;
}

struct ScaleOne {
    static constexpr double value = 1.0;
};
template <int N0>
struct ScaleOrtho {  // sqrt(2/N0)
    static constexpr double value = c_sqrt(2.0 / N0);
};
template <int N0>
constexpr float dc_scale() { return (float)c_sqrt(1.0 / N0); }

template <int I, int N, class F>
FDCT_HD void static_for(F &&f)
{
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}

template <int N, class SC>
FDCT_HD void dct4(const float (&v)[N], float (&V)[N]);

// out[k] = w_k * sum_n x[n] cos(pi (2n+1) k / (2N)),  w_0 = 1, w_k = SC
template <int N, class SC>
FDCT_HD void dct2(const float (&x)[N], float (&X)[N])
{
    if constexpr (N == 1) {
        X[0] = x[0];
    } else {
        constexpr int H = N / 2;
        float u[H], v[H], E[H], O[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            u[n] = x[n] + x[N - 1 - n];
            v[n] = x[n] - x[N - 1 - n];
        });
        dct2<H, SC>(u, E);
        dct4<H, SC>(v, O);
        static_for<0, H>([&](auto i) {
            constexpr int j = decltype(i)::value;
            X[2 * j] = E[j];
            X[2 * j + 1] = O[j];
        });
    }
}

// V[j] = SC * sum_n v[n] cos(pi (2n+1)(2j+1) / (4N))
template <int N, class SC>
FDCT_HD void dct4(const float (&v)[N], float (&V)[N])
{
    if constexpr (N == 1) {
        constexpr float c = (float)(SC::value * c_cos(kPi / 4.0));
        V[0] = v[0] * c;
    } else {
        constexpr int H = N / 2;
        float a[H], b[H], A[H], Bt[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            constexpr double th = (2.0 * n + 1.0) * kPi / (4.0 * N);
            constexpr double sg = (n % 2 == 0) ? 1.0 : -1.0;
            constexpr float c = (float)(SC::value * c_cos(th));
            constexpr float s = (float)(SC::value * c_sin(th));
            constexpr float cb = (float)(SC::value * sg * c_cos(th));
            constexpr float sb = (float)(SC::value * sg * c_sin(th));
            const float lo = v[n], hi = v[N - 1 - n];
            a[n] = fmaf(hi, s, lo * c);
            b[n] = fmaf(hi, cb, -(lo * sb));
        });
        dct2<H, ScaleOne>(a, A);
        dct2<H, ScaleOne>(b, Bt);
        V[0] = A[0];
        V[N - 1] = -Bt[0];
        static_for<1, H>([&](auto i) {
            constexpr int p = decltype(i)::value;
            V[2 * p - 1] = A[p] - Bt[H - p];
            V[2 * p] = A[p] + Bt[H - p];
        });
    }
}

// x[n] = sum_k w_k X[k] cos(pi (2n+1) k / (2N)),  w_0 = 1, w_k = SC   (transpose of dct2)
template <int N, class SC>
FDCT_HD void dct3(const float (&X)[N], float (&x)[N])
{
    if constexpr (N == 1) {
        x[0] = X[0];
    } else {
        constexpr int H = N / 2;
        float Xe[H], Xo[H], e[H], o[H];
        static_for<0, H>([&](auto i) {
            constexpr int j = decltype(i)::value;
            Xe[j] = X[2 * j];
            Xo[j] = X[2 * j + 1];
        });
        dct3<H, SC>(Xe, e);
        dct4<H, SC>(Xo, o);
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            x[n] = e[n] + o[n];
            x[N - 1 - n] = e[n] - o[n];
        });
    }
}

// Orthonormal DCT-II of x (in place): X[k] = a_k sum_n x[n] cos(pi (2n+1) k / (2N)).
template <int N>
FDCT_HD void dct2_ortho(float (&x)[N])
{
    float X[N];
    dct2<N, ScaleOrtho<N>>(x, X);
    X[0] *= dc_scale<N>();
    static_for<0, N>([&](auto i) { x[decltype(i)::value] = X[decltype(i)::value]; });
}

// Inverse of dct2_ortho (orthonormal DCT-III), in place.
template <int N>
FDCT_HD void dct3_ortho(float (&X)[N])
{
    float x[N];
    X[0] *= dc_scale<N>();
    dct3<N, ScaleOrtho<N>>(X, x);
    static_for<0, N>([&](auto i) { X[decltype(i)::value] = x[decltype(i)::value]; });
}

// ------------------------------------------------------------------------------------------------
// The same two transforms split so that the forward and the inverse share ONE copy of their
// multiplications.  DCT-II_N is a cascade of butterflies (sums go down, differences are the inputs of
// DCT-IV_{N/2}, DCT-IV_{N/4}, ..., DCT-IV_1) and DCT-III_N is the same DCT-IV blocks followed by the
// transposed cascade, so both are  [butterflies] o core  /  core o [butterflies]  with
//   core:  y[0] = dc * w[0],  y[H .. 2H) = DCT-IV_H(w[H .. 2H))  for H = 1, 2, 4, ..., N/2.
// Position p of w / y corresponds to coefficient core_index<N>(p).  A kernel that runs the core inside
// a rolled loop over its passes keeps a single copy of the (fully unrolled) DCT-IV code.
// ------------------------------------------------------------------------------------------------
template <int N>
constexpr int core_index(int p)
{
    if (p == 0) return 0;
    int h = 1;
    while (2 * h <= p) h *= 2;
    return (N / h) * (p - h) + N / (2 * h);
}
// inverse map: position of coefficient v
template <int N>
constexpr int core_pos(int v)
{
    for (int p = 0; p < N; ++p)
        if (core_index<N>(p) == v) return p;
    return -1;
}

template <int H, int N, class SC>
FDCT_HD void core_blocks(const float (&w)[N], float (&y)[N])
{
    float v[H], V[H];
    static_for<0, H>([&](auto i) { v[decltype(i)::value] = w[H + decltype(i)::value]; });
    dct4<H, SC>(v, V);
    static_for<0, H>([&](auto i) { y[H + decltype(i)::value] = V[decltype(i)::value]; });
    if constexpr (H > 1) core_blocks<H / 2, N, SC>(w, y);
}
template <int N>
FDCT_HD void dct_core_ortho(const float (&w)[N], float (&y)[N])
{
    y[0] = w[0] * dc_scale<N>();
    core_blocks<N / 2, N, ScaleOrtho<N>>(w, y);
}

// Forward butterflies: natural-order input x -> core input w.
template <int L, int N>
FDCT_HD void fwd_cascade(const float (&u)[L], float (&w)[N])
{
    if constexpr (L == 1) {
        w[0] = u[0];
    } else {
        constexpr int H = L / 2;
        float s[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            s[n] = u[n] + u[L - 1 - n];
            w[H + n] = u[n] - u[L - 1 - n];
        });
        fwd_cascade<H, N>(s, w);
    }
}
template <int N>
FDCT_HD void dct2_pre(const float (&x)[N], float (&w)[N])
{
    fwd_cascade<N, N>(x, w);
}

// Inverse butterflies: core output y -> natural-order output x.
template <int H, int N>
FDCT_HD void inv_cascade(const float (&e)[H], const float (&y)[N], float (&x)[N])
{
    if constexpr (H == N) {
        static_for<0, N>([&](auto i) { x[decltype(i)::value] = e[decltype(i)::value]; });
    } else {
        float f[2 * H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            f[n] = e[n] + y[H + n];
            f[2 * H - 1 - n] = e[n] - y[H + n];
        });
        inv_cascade<2 * H, N>(f, y, x);
    }
}
template <int N>
FDCT_HD void dct3_post(const float (&y)[N], float (&x)[N])
{
    float e[1] = {y[0]};
    inv_cascade<1, N>(e, y, x);
}

// ------------------------------------------------------------------------------------------------
// Two floats per operation.  sm_100 adds packed fp32 arithmetic (add / sub on a register pair, one issue
// slot for two results, each result rounded exactly like the scalar operation).  A kernel whose limit is
// instruction issue gains from it wherever two values go through the same addition at the same time:
//   * the two half-size DCT-II inside every DCT-IV work on independent vectors a and b: they run as ONE
//     transform over pairs (a[n], b[n]); nested DCT-IV blocks rotate each half of a pair by scalar
//     operations (the rotation constants would otherwise need register pairs of their own) and hand the
//     four resulting vectors on as two vectors of pairs;
//   * the butterfly cascades work on pairs of neighbouring elements, stored (x[2p], x[2p+1]) for even p
//     and swapped for odd p: the partner pair of pair j at a level of L elements is pair L/2-1-j, whose
//     swapped order is exactly the mirror image, and sums and differences come out in the same
//     alternating order for the next level.
// On the host the pair is two floats and the operations are the scalar ones (same results bit for bit).
// ------------------------------------------------------------------------------------------------
struct F2 {
#if defined(__CUDA_ARCH__)
    unsigned long long v;
#else
    float lo, hi;
#endif
};
FDCT_HD F2 f2_make(float lo, float hi)
{
    F2 r;
#if defined(__CUDA_ARCH__)
    asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
#else
    r.lo = lo;
    r.hi = hi;
#endif
    return r;
}
FDCT_HD float f2_lo(F2 a)
{
#if defined(__CUDA_ARCH__)
    float lo;
    asm("{\n\t.reg .b32 t;\n\tmov.b64 {%0, t}, %1;\n\t}" : "=f"(lo) : "l"(a.v));
    return lo;
#else
    return a.lo;
#endif
}
FDCT_HD float f2_hi(F2 a)
{
#if defined(__CUDA_ARCH__)
    float hi;
    asm("{\n\t.reg .b32 t;\n\tmov.b64 {t, %0}, %1;\n\t}" : "=f"(hi) : "l"(a.v));
    return hi;
#else
    return a.hi;
#endif
}
FDCT_HD F2 f2_add(F2 a, F2 b)
{
    F2 r;
#if defined(__CUDA_ARCH__)
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
#else
    r.lo = a.lo + b.lo;
    r.hi = a.hi + b.hi;
#endif
    return r;
}
FDCT_HD F2 f2_sub(F2 a, F2 b)
{
    F2 r;
#if defined(__CUDA_ARCH__)
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
#else
    r.lo = a.lo - b.lo;
    r.hi = a.hi - b.hi;
#endif
    return r;
}

FDCT_HD F2 f2_mul(F2 a, F2 b)
{
    F2 r;
#if defined(__CUDA_ARCH__)
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
#else
    r.lo = a.lo * b.lo;
    r.hi = a.hi * b.hi;
#endif
    return r;
}
FDCT_HD F2 f2_fma(F2 a, F2 b, F2 c)
{
    F2 r;
#if defined(__CUDA_ARCH__)
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v));
#else
    r.lo = fmaf(a.lo, b.lo, c.lo);
    r.hi = fmaf(a.hi, b.hi, c.hi);
#endif
    return r;
}

template <int N, class SC>
FDCT_HD void dct4v(const F2 (&v)[N], F2 (&V)[N]);

// DCT-II of two independent vectors at once (one in each half of the pairs); same scaling as dct2.
template <int N, class SC>
FDCT_HD void dct2v(const F2 (&x)[N], F2 (&X)[N])
{
    if constexpr (N == 1) {
        X[0] = x[0];
    } else {
        constexpr int H = N / 2;
        F2 u[H], v[H], E[H], O[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            u[n] = f2_add(x[n], x[N - 1 - n]);
            v[n] = f2_sub(x[n], x[N - 1 - n]);
        });
        dct2v<H, SC>(u, E);
        dct4v<H, SC>(v, O);
        static_for<0, H>([&](auto i) {
            constexpr int j = decltype(i)::value;
            X[2 * j] = E[j];
            X[2 * j + 1] = O[j];
        });
    }
}

// DCT-IV of two independent vectors at once; same scaling as dct4.
template <int N, class SC>
FDCT_HD void dct4v(const F2 (&v)[N], F2 (&V)[N])
{
    if constexpr (N == 1) {
        constexpr float c = (float)(SC::value * c_cos(kPi / 4.0));
        V[0] = f2_make(f2_lo(v[0]) * c, f2_hi(v[0]) * c);
    } else {
        constexpr int H = N / 2;
        F2 a[H], b[H], A[H], Bt[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            constexpr double th = (2.0 * n + 1.0) * kPi / (4.0 * N);
            constexpr double sg = (n % 2 == 0) ? 1.0 : -1.0;
            constexpr float c = (float)(SC::value * c_cos(th));
            constexpr float s = (float)(SC::value * c_sin(th));
            constexpr float cb = (float)(SC::value * sg * c_cos(th));
            constexpr float sb = (float)(SC::value * sg * c_sin(th));
            // both vectors turn by the same angle: packed multiply and multiply-add (rounded like the scalar forms)
            a[n] = f2_fma(v[N - 1 - n], f2_make(s, s), f2_mul(v[n], f2_make(c, c)));
            b[n] = f2_fma(v[N - 1 - n], f2_make(cb, cb), f2_mul(v[n], f2_make(-sb, -sb)));
        });
        dct2v<H, ScaleOne>(a, A);
        dct2v<H, ScaleOne>(b, Bt);
        V[0] = A[0];
        V[N - 1] = f2_make(-f2_lo(Bt[0]), -f2_hi(Bt[0]));
        static_for<1, H>([&](auto i) {
            constexpr int p = decltype(i)::value;
            V[2 * p - 1] = f2_sub(A[p], Bt[H - p]);
            V[2 * p] = f2_add(A[p], Bt[H - p]);
        });
    }
}

// dct4 with its two half-size DCT-II run as one transform over pairs (a[n], b[n]).
template <int N, class SC>
FDCT_HD void dct4_paired(const float (&v)[N], float (&V)[N])
{
    if constexpr (N <= 2) {
        dct4<N, SC>(v, V);
    } else {
        constexpr int H = N / 2;
        F2 ab[H], AB[H];
        static_for<0, H>([&](auto i) {
            constexpr int n = decltype(i)::value;
            constexpr double th = (2.0 * n + 1.0) * kPi / (4.0 * N);
            constexpr double sg = (n % 2 == 0) ? 1.0 : -1.0;
            constexpr float c = (float)(SC::value * c_cos(th));
            constexpr float s = (float)(SC::value * c_sin(th));
            constexpr float cb = (float)(SC::value * sg * c_cos(th));
            constexpr float sb = (float)(SC::value * sg * c_sin(th));
            const float lo = v[n], hi = v[N - 1 - n];
            ab[n] = f2_make(fmaf(hi, s, lo * c), fmaf(hi, cb, -(lo * sb)));
        });
        dct2v<H, ScaleOne>(ab, AB);
        V[0] = f2_lo(AB[0]);
        V[N - 1] = -f2_hi(AB[0]);
        static_for<1, H>([&](auto i) {
            constexpr int p = decltype(i)::value;
            V[2 * p - 1] = f2_lo(AB[p]) - f2_hi(AB[H - p]);
            V[2 * p] = f2_lo(AB[p]) + f2_hi(AB[H - p]);
        });
    }
}

template <int H, int N, class SC>
FDCT_HD void core_blocks_paired(const float (&w)[N], float (&y)[N])
{
    float v[H], V[H];
    static_for<0, H>([&](auto i) { v[decltype(i)::value] = w[H + decltype(i)::value]; });
    dct4_paired<H, SC>(v, V);
    static_for<0, H>([&](auto i) { y[H + decltype(i)::value] = V[decltype(i)::value]; });
    if constexpr (H > 1) core_blocks_paired<H / 2, N, SC>(w, y);
}
// dct_core_ortho with packed arithmetic (same results).
template <int N>
FDCT_HD void dct_core_ortho_paired(const float (&w)[N], float (&y)[N])
{
    y[0] = w[0] * dc_scale<N>();
    core_blocks_paired<N / 2, N, ScaleOrtho<N>>(w, y);
}

// Forward cascade on pairs of neighbours: a level of L elements is L/2 pairs, pair p = (e[2p], e[2p+1]) for even p and
// (e[2p+1], e[2p]) for odd p.
template <int L, int N>
FDCT_HD void fwd_cascade_paired(const F2 (&e)[L / 2], float (&w)[N])
{
    if constexpr (L == 2) {
        w[0] = f2_lo(e[0]) + f2_hi(e[0]);
        w[1] = f2_lo(e[0]) - f2_hi(e[0]);
    } else {
        constexpr int Q = L / 4;  // pairs of the next level
        F2 s[Q];
        static_for<0, Q>([&](auto i) {
            constexpr int j = decltype(i)::value;
            s[j] = f2_add(e[j], e[L / 2 - 1 - j]);
            const F2 d = f2_sub(e[j], e[L / 2 - 1 - j]);
            w[L / 2 + 2 * j] = (j % 2 == 0) ? f2_lo(d) : f2_hi(d);
            w[L / 2 + 2 * j + 1] = (j % 2 == 0) ? f2_hi(d) : f2_lo(d);
        });
        fwd_cascade_paired<L / 2, N>(s, w);
    }
}
template <int N>
FDCT_HD void dct2_pre_paired(const float (&x)[N], float (&w)[N])
{
    F2 e[N / 2];
    static_for<0, N / 2>([&](auto i) {
        constexpr int p = decltype(i)::value;
        e[p] = (p % 2 == 0) ? f2_make(x[2 * p], x[2 * p + 1]) : f2_make(x[2 * p + 1], x[2 * p]);
    });
    fwd_cascade_paired<N, N>(e, w);
}

// Inverse cascade on pairs: e holds H elements as H/2 pairs in the alternating order.
template <int H, int N>
FDCT_HD void inv_cascade_paired(const F2 (&e)[H / 2], const float (&y)[N], float (&x)[N])
{
    if constexpr (H == N) {
        static_for<0, N / 2>([&](auto i) {
            constexpr int p = decltype(i)::value;
            x[2 * p] = (p % 2 == 0) ? f2_lo(e[p]) : f2_hi(e[p]);
            x[2 * p + 1] = (p % 2 == 0) ? f2_hi(e[p]) : f2_lo(e[p]);
        });
    } else {
        F2 f[H];  // 2H elements
        static_for<0, H / 2>([&](auto i) {
            constexpr int j = decltype(i)::value;
            const F2 yy = (j % 2 == 0) ? f2_make(y[H + 2 * j], y[H + 2 * j + 1]) : f2_make(y[H + 2 * j + 1], y[H + 2 * j]);
            f[j] = f2_add(e[j], yy);
            f[H - 1 - j] = f2_sub(e[j], yy);
        });
        inv_cascade_paired<2 * H, N>(f, y, x);
    }
}
template <int N>
FDCT_HD void dct3_post_paired(const float (&y)[N], float (&x)[N])
{
    const F2 e[1] = {f2_make(y[0] + y[1], y[0] - y[1])};
    inv_cascade_paired<2, N>(e, y, x);
}
// dct2<N, SC> / dct3<N, SC> (any output scale SC, DC term unscaled) through the packed cascades and blocks: same
// results, about a third fewer instructions.
template <int N, class SC>
FDCT_HD void dct2_packed(const float (&x)[N], float (&X)[N])
{
    float w[N], y[N];
    dct2_pre_paired<N>(x, w);
    y[0] = w[0];
    core_blocks_paired<N / 2, N, SC>(w, y);
    static_for<0, N>([&](auto i) { X[core_index<N>(decltype(i)::value)] = y[decltype(i)::value]; });
}
template <int N, class SC>
FDCT_HD void dct3_packed(const float (&X)[N], float (&x)[N])
{
    float w[N], y[N];
    static_for<0, N>([&](auto i) { w[decltype(i)::value] = X[core_index<N>(decltype(i)::value)]; });
    y[0] = w[0];
    core_blocks_paired<N / 2, N, SC>(w, y);
    dct3_post_paired<N>(y, x);
}

// The same with the result left in pairs: xp[p] = (x[2p], x[2p+1]) for even p, (x[2p+1], x[2p]) for odd p.
template <int H, int N>
FDCT_HD void inv_cascade_pairs(const F2 (&e)[H / 2], const float (&y)[N], F2 (&xp)[N / 2])
{
    if constexpr (H == N) {
        static_for<0, N / 2>([&](auto i) { xp[decltype(i)::value] = e[decltype(i)::value]; });
    } else {
        F2 f[H];
        static_for<0, H / 2>([&](auto i) {
            constexpr int j = decltype(i)::value;
            const F2 yy = (j % 2 == 0) ? f2_make(y[H + 2 * j], y[H + 2 * j + 1]) : f2_make(y[H + 2 * j + 1], y[H + 2 * j]);
            f[j] = f2_add(e[j], yy);
            f[H - 1 - j] = f2_sub(e[j], yy);
        });
        inv_cascade_pairs<2 * H, N>(f, y, xp);
    }
}
template <int N>
FDCT_HD void dct3_post_pairs(const float (&y)[N], F2 (&xp)[N / 2])
{
    const F2 e[1] = {f2_make(y[0] + y[1], y[0] - y[1])};
    inv_cascade_pairs<2, N>(e, y, xp);
}
// Position of element v in the "pair order" (neighbours of odd pairs swapped); its own inverse.
constexpr int pair_order(int v) { return v ^ ((v >> 1) & 1); }

}  // namespace fdct
