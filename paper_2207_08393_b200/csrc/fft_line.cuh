// Multi-stage line FFT held in registers, with the stage hand-over through shared memory.
//
// A line of N = R0*R1*R2 points is transformed in up to three stages of in-register butterflies.
//   first stage : thread j (0 <= j < N/R0) holds x[j + (N/R0) m], m < R0        ("n-distribution")
//   last stage  : thread j (0 <= j < N/RL) holds X[j + (N/RL) k], k < RL        ("k-distribution")
// The forward transform goes from the n- to the k-distribution, the inverse mirrors it stage by
// stage (conjugated butterflies and twiddles, reversed order), so a pointwise operation in
// k-space sits between them without any reordering.  Transforms are raw: no scaling, no centring.
//
// Several lines are processed per thread block.  ROW mode: the line is contiguous in memory and
// consecutive threads take consecutive butterflies of one line.  COL mode: the line is strided and
// consecutive threads take the same butterfly of consecutive lines (contiguous in memory).
#pragma once
#include "fft_radix.cuh"

namespace gleam {

constexpr int cmax(int a, int b) { return a > b ? a : b; }
constexpr int odd_up(int a) { return (a % 2 == 0) ? a + 1 : a; }

template <int N_, int R0_, int R1_ = 1, int R2_ = 1>
struct Plan {
    static constexpr int N = N_, R0 = R0_, R1 = R1_, R2 = R2_;
    static_assert(R0 * R1 * R2 == N, "radices must multiply to N");
    static constexpr int S = (R2 > 1) ? 3 : (R1 > 1 ? 2 : 1);
    static constexpr int RL = (S == 3) ? R2 : (S == 2 ? R1 : R0);
    static constexpr int N1 = N / R0;              // sub-length after the first stage
    static constexpr int N2 = N1 / R1;             // sub-length after the second stage (S == 3)
    static constexpr int BF0 = N / R0, BF1 = N / R1, BFL = N / RL;   // butterflies per line and stage
    static constexpr int MAXBF = (S == 3) ? cmax(BF0, cmax(BF1, BFL)) : cmax(BF0, BFL);
    static constexpr int LS1 = odd_up(N1), LS2 = odd_up(N2);
    static constexpr int SM_A = (S >= 2) ? R0 * LS1 : 0;
    static constexpr int SM_B = (S == 3) ? R0 * R1 * LS2 : 0;
    static constexpr int BUF = cmax(SM_A, SM_B);   // one exchange buffer (elements)
    static constexpr int LSZ = 2 * BUF;            // two buffers per line
};

// exp(-2 pi i e / N), e = 0..N-1, evaluated at compile time in double precision and stored as a
// device-resident constant table (a few KB per length, read through L1).
template <int N> struct RootTable { cf v[N]; };
template <int N> constexpr RootTable<N> make_root_table() {
    RootTable<N> t{};
    for (int e = 0; e < N; ++e) t.v[e] = cf{float(ct::cos2pi(e, N)), float(-ct::sin2pi(e, N))};
    return t;
}
template <int N> __device__ const RootTable<N> g_roots = make_root_table<N>();

template <int N> __device__ __forceinline__ cf unit_root_fwd(int e) { return g_roots<N>.v[e]; }

template <class P, bool COL, int L>
struct LineFFT {
    static constexpr int N = P::N, R0 = P::R0, R1 = P::R1, RL = P::RL, S = P::S;
    static constexpr int THREADS = ((L * P::MAXBF + 31) / 32) * 32;
    static constexpr int SMEM_ELEMS = L * P::LSZ + 1;
    static constexpr size_t SMEM_BYTES = sizeof(cf) * SMEM_ELEMS;

    // which line / butterfly a thread owns in each stage
    struct Ids {
        int l0, j0, l1, j1, lL, jL;
        bool a0, a1, aL;
    };
    __device__ __forceinline__ static void split(int tid, int bf, int& l, int& j, bool& act) {
        if (COL) { l = tid % L; j = tid / L; }
        else     { l = tid / bf; j = tid % bf; }
        act = (tid < L * bf);
    }
    __device__ __forceinline__ static Ids ids(int tid) {
        Ids d;
        split(tid, P::BF0, d.l0, d.j0, d.a0);
        split(tid, P::BFL, d.lL, d.jL, d.aL);
        if (S == 3) split(tid, P::BF1, d.l1, d.j1, d.a1);
        else { d.l1 = 0; d.j1 = 0; d.a1 = false; }
        return d;
    }
    __device__ __forceinline__ static int sidx(int l, int off) {
        return COL ? (off * L + l) : (l * P::LSZ + off);
    }

    struct Tw {
        cf t0[R0];      // exp(-2 pi i j0 k0 / N)
        cf t1[R1];      // exp(-2 pi i t k1 / N1)   (three-stage plans)
    };
    __device__ __forceinline__ static void make_tw(const Ids& d, Tw& tw) {
        if (S >= 2) {
#pragma unroll
            for (int k = 0; k < R0; ++k) tw.t0[k] = unit_root_fwd<N>((d.j0 * k) % N);
        }
        if (S == 3) {
            const int t = d.j1 % P::N2;
#pragma unroll
            for (int k = 0; k < R1; ++k) tw.t1[k] = unit_root_fwd<(P::S == 3 ? P::N1 : 1)>(P::S == 3 ? (t * k) % P::N1 : 0);
        }
    }

    // v: n-distribution of the first-stage thread; u: k-distribution of the last-stage thread
    // flip = 1 swaps the two exchange buffers of a two-stage plan.  A loop that calls only forward()
    // (or only inverse()) must alternate flip from one call to the next: with a single barrier per
    // call, the buffer written now must not be the one other threads may still be reading.
    __device__ __forceinline__ static void forward(cf (&v)[R0], cf (&u)[RL], const Tw& tw, const Ids& d, cf* sm,
                                                   int flip = 0) {
        cf* X = sm + ((S == 2 && flip) ? (COL ? L * P::BUF : P::BUF) : 0);
        cf* Y = sm + (COL ? L * P::BUF : P::BUF);
        forward_xy(v, u, tw, d, X, Y);
    }
    // forward with explicit exchange buffers (two-stage plans use X only)
    __device__ __forceinline__ static void forward_xy(cf (&v)[R0], cf (&u)[RL], const Tw& tw, const Ids& d, cf* X,
                                                      cf* Y) {
        if (S == 1) {
            Dft<R0, -1>::run(v);
#pragma unroll
            for (int k = 0; k < RL; ++k) u[k] = v[k % R0];
            return;
        }
        if (d.a0) {
            Dft<R0, -1>::run(v);
#pragma unroll
            for (int k = 0; k < R0; ++k) {
                cf t = (k == 0) ? v[0] : cmul(v[k], tw.t0[k]);
                X[sidx(d.l0, k * P::LS1 + d.j0)] = t;
            }
        }
        __syncthreads();
        if (S == 3) {
            if (d.a1) {
                const int q = d.j1 / P::N2, t = d.j1 % P::N2;
                cf w[R1];
#pragma unroll
                for (int m = 0; m < R1; ++m) w[m] = X[sidx(d.l1, q * P::LS1 + t + P::N2 * m)];
                Dft<R1, -1>::run(w);
#pragma unroll
                for (int k = 0; k < R1; ++k) {
                    cf r = (k == 0) ? w[0] : cmul(w[k], tw.t1[k]);
                    Y[sidx(d.l1, (k * R0 + q) * P::LS2 + t)] = r;
                }
            }
            __syncthreads();
            if (d.aL) {
#pragma unroll
                for (int m = 0; m < RL; ++m) u[m] = Y[sidx(d.lL, d.jL * P::LS2 + m)];
                Dft<RL, -1>::run(u);
            }
        } else {
            if (d.aL) {
#pragma unroll
                for (int m = 0; m < RL; ++m) u[m] = X[sidx(d.lL, d.jL * P::LS1 + m)];
                Dft<RL, -1>::run(u);
            }
        }
    }

    // mirror image of forward(): u (k-distribution) -> v (n-distribution), unscaled inverse.
    // Buffer use: two-stage plans exchange through Y (X may still be read by forward());
    // three-stage plans go through X then Y.
    __device__ __forceinline__ static void inverse(cf (&u)[RL], cf (&v)[R0], const Tw& tw, const Ids& d, cf* sm,
                                                   int flip = 0) {
        cf* X = sm;
        cf* Y = sm + ((S == 2 && flip) ? 0 : (COL ? L * P::BUF : P::BUF));
        inverse_xy(u, v, tw, d, X, Y);
    }
    // inverse with explicit exchange buffers (two-stage plans use Y only)
    __device__ __forceinline__ static void inverse_xy(cf (&u)[RL], cf (&v)[R0], const Tw& tw, const Ids& d, cf* X,
                                                      cf* Y) {
        if (S == 1) {
#pragma unroll
            for (int k = 0; k < R0; ++k) v[k] = u[k % RL];
            Dft<R0, +1>::run(v);
            return;
        }
        if (S == 3) {
            if (d.aL) {
                Dft<RL, +1>::run(u);
#pragma unroll
                for (int m = 0; m < RL; ++m) X[sidx(d.lL, d.jL * P::LS2 + m)] = u[m];
            }
            __syncthreads();
            if (d.a1) {
                const int q = d.j1 / P::N2, t = d.j1 % P::N2;
                cf w[R1];
#pragma unroll
                for (int k = 0; k < R1; ++k) {
                    cf r = X[sidx(d.l1, (k * R0 + q) * P::LS2 + t)];
                    w[k] = (k == 0) ? r : cmulc(r, tw.t1[k]);
                }
                Dft<R1, +1>::run(w);
#pragma unroll
                for (int m = 0; m < R1; ++m) Y[sidx(d.l1, q * P::LS1 + t + P::N2 * m)] = w[m];
            }
            __syncthreads();
        } else {
            if (d.aL) {
                Dft<RL, +1>::run(u);
#pragma unroll
                for (int m = 0; m < RL; ++m) Y[sidx(d.lL, d.jL * P::LS1 + m)] = u[m];
            }
            __syncthreads();
        }
        if (d.a0) {
#pragma unroll
            for (int k = 0; k < R0; ++k) {
                cf r = Y[sidx(d.l0, k * P::LS1 + d.j0)];
                v[k] = (k == 0) ? r : cmulc(r, tw.t0[k]);
            }
            Dft<R0, +1>::run(v);
        }
    }
};

}  // namespace gleam
