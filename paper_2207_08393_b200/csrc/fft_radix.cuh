// In-register DFT butterflies of compile-time radix with compile-time twiddle constants.
//
// Every routine computes the raw (unscaled, uncentred) DFT
//     X[k] = sum_n x[n] * exp(DIR * 2 pi i * n k / R),   DIR = -1 (forward) or +1 (inverse),
// in place on a register array, natural order in and out.  Radices: 2 and 4 are written out,
// odd primes use the symmetric direct form (pairs x[m] +- x[R-m], real cosine / sine sums),
// composites with coprime factors use the prime-factor index maps (no inner twiddles), the others
// are split Cooley-Tukey style with the inner twiddles folded in as constants.
#pragma once
#include <cuda_runtime.h>

namespace gleam {

typedef float2 cf;

#define GLEAM_HD __host__ __device__ __forceinline__

// ------------------------------------------------------------------------------------------
// compile-time cos / sin of 2 pi k / n  (double precision Taylor series after octant reduction)
// ------------------------------------------------------------------------------------------
namespace ct {
constexpr double PI = 3.14159265358979323846264338327950288;

constexpr double taylor_sin(double x) {   // |x| <= pi/4
    double term = x, sum = x;
    const double x2 = x * x;
    for (int i = 1; i < 14; ++i) { term *= -x2 / double((2 * i) * (2 * i + 1)); sum += term; }
    return sum;
}
constexpr double taylor_cos(double x) {
    double term = 1.0, sum = 1.0;
    const double x2 = x * x;
    for (int i = 1; i < 14; ++i) { term *= -x2 / double((2 * i - 1) * (2 * i)); sum += term; }
    return sum;
}
// cos(2 pi k / n) and sin(2 pi k / n) for any integer k, n > 0
constexpr double cos2pi(long long k, long long n) {
    k %= n; if (k < 0) k += n;
    // fold to [0, n/2]
    if (2 * k > n) k = n - k;                     // cos even around pi
    // now angle in [0, pi]; fold to [0, pi/2]
    bool neg = false;
    long long kk = k, nn = n;
    if (4 * kk > nn) { kk = nn - 2 * kk; nn = 2 * nn; neg = true; }   // cos(pi - a) = -cos a : a = 2pi*(n/2-k)/n = 2pi*(n-2k)/(2n)
    // angle = 2 pi kk / nn in [0, pi/2]
    double r = 0.0;
    if (8 * kk <= nn) r = taylor_cos(2.0 * PI * double(kk) / double(nn));
    else r = taylor_sin(2.0 * PI * double(nn - 4 * kk) / double(4 * nn));  // cos a = sin(pi/2 - a)
    return neg ? -r : r;
}
constexpr double sin2pi(long long k, long long n) {
    // sin(a) = cos(a - pi/2) = cos(2 pi (4k - n) / (4n))
    return cos2pi(4 * k - n, 4 * n);
}
}  // namespace ct

// ------------------------------------------------------------------------------------------
// complex helpers
// ------------------------------------------------------------------------------------------
// Complex add / subtract / real-scaled accumulate use the packed two-lane FP32 instructions of
// sm_100 (one issue slot for both components); rounding is identical to the scalar forms.
GLEAM_HD cf cadd(cf a, cf b) {
#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ >= 1000)
    return __fadd2_rn(a, b);
#else
    return make_float2(a.x + b.x, a.y + b.y);
#endif
}
GLEAM_HD cf csub(cf a, cf b) {
#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ >= 1000)
    return __ffma2_rn(b, make_float2(-1.f, -1.f), a);
#else
    return make_float2(a.x - b.x, a.y - b.y);
#endif
}
// acc + c * a  with a real constant c
GLEAM_HD cf caxpy(float c, cf a, cf acc) {
#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ >= 1000)
    return __ffma2_rn(make_float2(c, c), a, acc);
#else
    return make_float2(fmaf(c, a.x, acc.x), fmaf(c, a.y, acc.y));
#endif
}
GLEAM_HD cf cmul(cf a, cf b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
GLEAM_HD cf cmulc(cf a, cf b) { return make_float2(a.x * b.x + a.y * b.y, a.y * b.x - a.x * b.y); }  // a * conj(b)
GLEAM_HD cf cscale(cf a, float s) { return make_float2(a.x * s, a.y * s); }
// a * (DIR>0 ? +i : -i)
template <int DIR> GLEAM_HD cf mul_i_dir(cf a) {
    return DIR > 0 ? make_float2(-a.y, a.x) : make_float2(a.y, -a.x);
}

// multiply by the constant exp(DIR 2 pi i K / N), trivial cases resolved at compile time
template <int K_, int N, int DIR> GLEAM_HD cf mul_tw(cf a) {
    constexpr int K = ((K_ % N) + N) % N;
    if constexpr (K == 0) return a;
    else if constexpr (2 * K == N) return make_float2(-a.x, -a.y);
    else if constexpr (4 * K == N) return mul_i_dir<DIR>(a);
    else if constexpr (4 * K == 3 * N) return mul_i_dir<-DIR>(a);
    else {
        constexpr float c = float(ct::cos2pi(K, N));
        constexpr float s = float(DIR * ct::sin2pi(K, N));
        if constexpr (8 * K == N || 8 * K == 3 * N || 8 * K == 5 * N || 8 * K == 7 * N) {
            // |c| == |s| = 1/sqrt2
            constexpr float h = 0.70710678118654752440f;
            constexpr float sc = c > 0 ? 1.f : -1.f, ss = s > 0 ? 1.f : -1.f;
            // (x + i y)(sc + i ss) h
            return make_float2((sc * a.x - ss * a.y) * h, (ss * a.x + sc * a.y) * h);
        } else {
            return make_float2(a.x * c - a.y * s, a.x * s + a.y * c);
        }
    }
}

// ------------------------------------------------------------------------------------------
// helpers for compile-time loops
// ------------------------------------------------------------------------------------------
template <int I> struct IC { static constexpr int value = I; };
template <int B, int E, class F> GLEAM_HD void static_for(F&& f) {
    if constexpr (B < E) { f(IC<B>{}); static_for<B + 1, E>(f); }
}

constexpr int smallest_odd_factor(int r) {
    for (int p = 3; p * p <= r; p += 2) if (r % p == 0) return p;
    return r;
}
constexpr int ct_factor(int r) {     // outer factor A of the split R = A * B
    return (r % 4 == 0) ? 4 : (r % 2 == 0) ? 2 : smallest_odd_factor(r);
}
constexpr bool is_prime_like(int r) { return r == 2 || r == 4 || (r % 2 == 1 && smallest_odd_factor(r) == r); }

template <int R, int DIR> struct Dft;

template <int DIR> struct Dft<1, DIR> { static GLEAM_HD void run(cf (&)[1]) {} };

template <int DIR> struct Dft<2, DIR> {
    static GLEAM_HD void run(cf (&v)[2]) {
        const cf a = v[0], b = v[1];
        v[0] = cadd(a, b); v[1] = csub(a, b);
    }
};

template <int DIR> struct Dft<4, DIR> {
    static GLEAM_HD void run(cf (&v)[4]) {
        const cf s02 = cadd(v[0], v[2]), d02 = csub(v[0], v[2]);
        const cf s13 = cadd(v[1], v[3]), d13 = csub(v[1], v[3]);
        v[0] = cadd(s02, s13); v[2] = csub(s02, s13);
        // v1 = d02 + (DIR i) d13,  v3 = d02 - (DIR i) d13   (component-wise: no register swap needed)
        if (DIR > 0) {
            v[1] = make_float2(d02.x - d13.y, d02.y + d13.x);
            v[3] = make_float2(d02.x + d13.y, d02.y - d13.x);
        } else {
            v[1] = make_float2(d02.x + d13.y, d02.y - d13.x);
            v[3] = make_float2(d02.x - d13.y, d02.y + d13.x);
        }
    }
};

// odd prime P: symmetric direct evaluation
template <int P, int DIR> struct DftPrime {
    static GLEAM_HD void run(cf (&v)[P]) {
        constexpr int H = (P - 1) / 2;
        cf a[H], b[H];
        cf x0 = v[0];
        cf sum = x0;
        static_for<0, H>([&](auto mi) {
            constexpr int m = decltype(mi)::value + 1;
            a[m - 1] = cadd(v[m], v[P - m]);
            b[m - 1] = csub(v[m], v[P - m]);
            sum = cadd(sum, a[m - 1]);
        });
        v[0] = sum;
        static_for<0, H>([&](auto ki) {
            constexpr int k = decltype(ki)::value + 1;
            cf C = x0, D = make_float2(0.f, 0.f);
            static_for<0, H>([&](auto mi) {
                constexpr int m = decltype(mi)::value + 1;
                constexpr float c = float(ct::cos2pi((long long)k * m, P));
                constexpr float s = float(ct::sin2pi((long long)k * m, P));
                C = caxpy(c, a[m - 1], C);
                D = caxpy(s, b[m - 1], D);
            });
            // X[k] = C + DIR * i * D ,  X[P-k] = C - DIR * i * D
            if (DIR > 0) {
                v[k] = make_float2(C.x - D.y, C.y + D.x);
                v[P - k] = make_float2(C.x + D.y, C.y - D.x);
            } else {
                v[k] = make_float2(C.x + D.y, C.y - D.x);
                v[P - k] = make_float2(C.x - D.y, C.y + D.x);
            }
        });
    }
};

// composite R = A * B, decimation in time:  n = A n2 + n1,  k = k2 + B k1
template <int R, int DIR> struct DftComposite {
    static constexpr int A = ct_factor(R);
    static constexpr int B = R / A;
    static GLEAM_HD void run(cf (&v)[R]) {
        cf y[A][B];
        static_for<0, A>([&](auto n1i) {
            constexpr int n1 = decltype(n1i)::value;
            cf t[B];
            static_for<0, B>([&](auto n2i) { constexpr int n2 = decltype(n2i)::value; t[n2] = v[A * n2 + n1]; });
            Dft<B, DIR>::run(t);
            static_for<0, B>([&](auto k2i) {
                constexpr int k2 = decltype(k2i)::value;
                y[n1][k2] = mul_tw<n1 * k2, R, DIR>(t[k2]);
            });
        });
        static_for<0, B>([&](auto k2i) {
            constexpr int k2 = decltype(k2i)::value;
            cf t[A];
            static_for<0, A>([&](auto n1i) { constexpr int n1 = decltype(n1i)::value; t[n1] = y[n1][k2]; });
            Dft<A, DIR>::run(t);
            static_for<0, A>([&](auto k1i) { constexpr int k1 = decltype(k1i)::value; v[k2 + B * k1] = t[k1]; });
        });
    }
};

// composite R = A * B with coprime factors (6, 10, 12, 15, 20, ...): prime-factor index maps,
//   n = (B n1 + A n2) mod R,   k = the residue with k mod A = k1 and k mod B = k2,
// turn the transform into A-point and B-point transforms with no twiddle factors in between
// (W_R^{B n1 k} = W_A^{n1 k1},  W_R^{A n2 k} = W_B^{n2 k2}).
constexpr int ct_gcd(int a, int b) { return b == 0 ? a : ct_gcd(b, a % b); }
constexpr int crt_index(int k1, int A, int k2, int B) {
    for (int k = 0; k < A * B; ++k) if (k % A == k1 && k % B == k2) return k;
    return 0;
}
template <int R, int DIR> struct DftCoprime {
    static constexpr int A = ct_factor(R);
    static constexpr int B = R / A;
    static GLEAM_HD void run(cf (&v)[R]) {
        cf y[A][B];
        static_for<0, A>([&](auto n1i) {
            constexpr int n1 = decltype(n1i)::value;
            cf t[B];
            static_for<0, B>([&](auto n2i) { constexpr int n2 = decltype(n2i)::value; t[n2] = v[(B * n1 + A * n2) % R]; });
            Dft<B, DIR>::run(t);
            static_for<0, B>([&](auto k2i) { constexpr int k2 = decltype(k2i)::value; y[n1][k2] = t[k2]; });
        });
        static_for<0, B>([&](auto k2i) {
            constexpr int k2 = decltype(k2i)::value;
            cf t[A];
            static_for<0, A>([&](auto n1i) { constexpr int n1 = decltype(n1i)::value; t[n1] = y[n1][k2]; });
            Dft<A, DIR>::run(t);
            static_for<0, A>([&](auto k1i) { constexpr int k1 = decltype(k1i)::value; v[crt_index(k1, A, k2, B)] = t[k1]; });
        });
    }
};

template <int R, int DIR> struct Dft {
    static GLEAM_HD void run(cf (&v)[R]) {
        if constexpr (R % 2 == 1 && smallest_odd_factor(R) == R) DftPrime<R, DIR>::run(v);
        else if constexpr (ct_gcd(ct_factor(R), R / ct_factor(R)) == 1) DftCoprime<R, DIR>::run(v);
        else DftComposite<R, DIR>::run(v);
    }
};

}  // namespace gleam
