// Kernels of the data-consistency step  out = x - eta * A^H (A x - y),  A = Omega F S  (Eq. 3 of
// the GLEAM paper with eta = 2t; sensing model Eq. 1) and of its vector-Jacobian product.
//
// All transforms inside the kernels are raw DFTs.  Centring and orthonormal scaling of F are moved
// into the k-space tables: with the shift sh(k) = (k + N/2) mod N per transformed axis,
//     A^H A   = S^H  Fraw^H  diag( M[sh(k)]^2 / N )  Fraw  S
//     A^H y   = S^H  Fraw^H  ( g (-1)^{sh(k)} M[sh(k)] y[sh(k)] / sqrt(N) ),   g = prod (-1)^{N_a/2}
// (even extents only).
//
// ROW kernels transform the contiguous axis n2 and carry the image-side work (sensitivity
// multiply on the way in, conjugate-sensitivity coil sum in registers on the way out).
// COL kernels transform a strided axis in place on a workspace, or turn y into the table z.
#pragma once
#include "fft_line.cuh"
#include <stdint.h>

#include "launch_overlap.cuh"

namespace gleam {

enum RowMode { ROW_FUSED = 0, ROW_FWD = 1, ROW_INV = 2 };
enum ColMode { COL_Z = 0, COL_MID_SEP = 1, COL_MID_FULL = 2, COL_FWD = 3, COL_INV = 4, COL_GRADY = 5 };

struct RowArgs {
    const cf* x;        // image-domain input (B,T,n0,n1,n2)
    const cf* sens;     // (B,C,[T],n0,n1,n2)
    cf* out;            // (B,T,n0,n1,n2)
    const float* mask;  // ROW_FUSED: readout-invariant mask (B,T,n2)
    const cf* z;        // ROW_FUSED: compact table of shifted, signed, masked R^H y: (B,C,T,n1,[rank < n2]); may be null
    const int* zidx;    // fallback row kernel with z: (B,T,n2) rank of a raw k index among the sampled ones, -1 if unsampled
    cf* W;              // workspace (unit, rpb, n2)
    float eta;
    int C, T, Ts;       // coils, frames, sens frames (T or 1)
    int rpb;            // rows of this launch per (b,t)
    int row0;           // first row of this launch inside the full image rows
    int RPB;            // rows of a full image (n0*n1)
    long long nrows;    // B*T*rpb
    double* dot_rows;   // ROW_FUSED (warp-resident form): if not null, Re<x, out> of every image row, (B*T*rpb)
    // Two-real-channel layout (B, 2, T, n0, n1, n2) float32 of the image-side arrays (the form the learned
    // prior takes and returns): real index of complex element e of example b = e + b * plane, the imaginary
    // part `plane` further on (plane = T * n0 * n1 * n2).
    int x_planar, out_planar;
    long long plane;
    // Normal-equations form of the step: when not null (only with z == null), the image A^H y (B,T,n0,n1,n2),
    // complex interleaved; the kernels that write `out` then store x - eta * (sum - aty).
    const cf* aty;
};

// Start value of the coil sum of image element e: minus the given A^H y, if there is one.  Taking it as the
// start value puts its load at the beginning of the coil loop, where its latency costs nothing, and needs no
// register of its own.
__device__ __forceinline__ cf coil_sum_start(const cf* aty, long long e) {
    if (aty == nullptr) return make_float2(0.f, 0.f);
    const cf t = aty[e];
    return make_float2(-t.x, -t.y);
}

// image-side element e (complex-element offset in the (B,T,V) array) of example b, in either layout
__device__ __forceinline__ cf load_image(const cf* x, long long e, int planar, int b, long long plane) {
    if (!planar) return x[e];
    const float* xf = reinterpret_cast<const float*>(x) + e + (long long)b * plane;
    return make_float2(xf[0], xf[plane]);
}
__device__ __forceinline__ void store_image(cf* out, long long e, cf v, int planar, int b, long long plane) {
    if (!planar) { out[e] = v; return; }
    float* of = reinterpret_cast<float*>(out) + e + (long long)b * plane;
    of[0] = v.x; of[plane] = v.y;
}

struct ColArgs {
    cf* W;              // in-place data (COL_MID_*, COL_FWD, COL_INV)
    const cf* y;        // COL_Z input / COL_MID_FULL measurements (B,C,T,V)
    cf* z;              // COL_Z output: compact table (unit, n_ro, [rank < pe])
    const cf* zin;      // COL_MID_SEP: compact z table (unit, n0, [rank < n1 n2])
    const int* zidx;    // (B,T,pe): rank of a raw k position among the sampled ones, -1 if unsampled
    const int* zlist;   // (B,T,pe): sampled source positions p (unshifted), by rank
    const int* zcount;  // (B,T)
    const float* m2c;   // (B,T,pe): squared mask weight of the sampled positions, by rank
    const int* zstart;  // row-tile path: (B,T,33) first rank of each ky-mod-RY group (null otherwise)
    const float* mask;  // COL_Z, COL_MID_SEP: readout-invariant mask; COL_MID_FULL: full mask (B,T,V)
    int es;             // element stride of the transformed axis = lines per outer index
    long long nouter;   // outer indices
    int C, T;
    int rank, n0, n1, n2;
    int G, i0_start;    // COL_MID_SEP chunk: slabs in the chunk, first slab
    int ztiles;         // COL_Z: blocks launched per outer index (they stride over the tiles of ranks)
    float scale;        // COL_Z: g_ro g_pe / sqrt(N_ro N_pe);  COL_MID_FULL: g / sqrt(Ntot)
    float scale2;       // COL_MID_FULL: 1 / Ntot;  COL_MID_SEP: 1 / (n1 n2)
    cf* ky_out;         // COL_GRADY: k-space output (B,C,T,V), written at the centred positions
    int mask_pe;        // COL_GRADY: 0 = full mask (B,T,V); else the mask is readout-invariant with this many entries per image
};

constexpr int COLZ_SELF_MAX = 1024;   // COL_Z ranks a mask row of at most this many positions by itself

__device__ __forceinline__ int shift_half(int k, int n) { int h = n >> 1; return k >= n - h ? k - (n - h) : k + h; }

// --------------------------------------------------------------------------------------------
// ROW kernel: L contiguous lines per block, all coils looped inside the block.
// --------------------------------------------------------------------------------------------
template <class P, int L, int MODE>
__global__ void __launch_bounds__(LineFFT<P, false, L>::THREADS)
row_kernel(const RowArgs a) {
    using E = LineFFT<P, false, L>;
    constexpr int N = P::N, R0 = P::R0, RL = P::RL;
    extern __shared__ float2 smem[];
    const typename E::Ids d = E::ids(threadIdx.x);
    typename E::Tw tw;
    E::make_tw(d, tw);

    // first-stage identity of this thread
    const long long r0 = (long long)blockIdx.x * L + d.l0;
    const bool act0 = d.a0 && r0 < a.nrows;
    const long long bt0 = act0 ? r0 / a.rpb : 0;
    const int ri0 = act0 ? (int)(r0 % a.rpb) : 0;
    const int b0 = (int)(bt0 / a.T), t0 = (int)(bt0 % a.T);
    // last-stage identity
    const long long rL = (long long)blockIdx.x * L + d.lL;
    const bool actL = d.aL && rL < a.nrows;
    const long long btL = actL ? rL / a.rpb : 0;
    const int riL = actL ? (int)(rL % a.rpb) : 0;
    const int bL = (int)(btL / a.T), tL = (int)(btL % a.T);

    const long long x_off = ((long long)bt0 * a.RPB + a.row0 + ri0) * N;
    cf xv[R0], acc[R0];
    if (MODE != ROW_FWD) {
#pragma unroll
        for (int m = 0; m < R0; ++m) acc[m] = act0 ? coil_sum_start(a.aty, x_off + d.j0 + P::BF0 * m) : make_float2(0.f, 0.f);
    }
    if (MODE != ROW_INV) {
        if (act0) {
#pragma unroll
            for (int m = 0; m < R0; ++m) xv[m] = load_image(a.x, x_off + d.j0 + P::BF0 * m, a.x_planar, b0, a.plane);
        }
    }
    float m2v[RL];
    if (MODE == ROW_FUSED) {
        if (actL) {
#pragma unroll
            for (int k = 0; k < RL; ++k) {
                const float mv = a.mask[btL * N + shift_half(d.jL + P::BFL * k, N)];
                m2v[k] = mv * mv * (1.0f / N);
            }
        }
    }

    // per-coil strides (elements); the loads of coil c+1 are issued before the arithmetic of coil c
    const long long s_stride = (long long)a.Ts * a.RPB * N;
    const long long s_base = (((long long)(b0 * a.C) * a.Ts + (a.Ts > 1 ? t0 : 0)) * a.RPB + a.row0 + ri0) * N + d.j0;
    const long long k_stride = (long long)a.T * ((MODE == ROW_FUSED) ? a.RPB : a.rpb) * N;
    const long long k_base = (MODE == ROW_FUSED)
        ? (((long long)(bL * a.C) * a.T + tL) * a.RPB + a.row0 + riL) * N + d.jL
        : (((long long)(bL * a.C) * a.T + tL) * a.rpb + riL) * N + d.jL;
    const bool use_z = (MODE == ROW_FUSED) && (a.z != nullptr);

    cf s_cur[R0], s_nxt[R0];      // sensitivities of this / the next coil (n-distribution)
    cf k_cur[RL], k_nxt[RL];      // z table (ROW_FUSED) or workspace (ROW_INV) values (k-distribution)
    auto load_s = [&](cf (&dst)[R0], int c) {
        if (act0) {
#pragma unroll
            for (int m = 0; m < R0; ++m) dst[m] = a.sens[s_base + c * s_stride + P::BF0 * m];
        }
    };
    auto load_k = [&](cf (&dst)[RL], int c) {
        if (actL) {
            const cf* src = (MODE == ROW_FUSED) ? a.z : a.W;
#pragma unroll
            for (int k = 0; k < RL; ++k) dst[k] = src[k_base + c * k_stride + P::BFL * k];
        }
    };
    load_s(s_cur, 0);
    if (MODE == ROW_INV) load_k(k_cur, 0);
    int zi[RL];
    if (use_z && actL) {
#pragma unroll
        for (int k = 0; k < RL; ++k) zi[k] = a.zidx[btL * N + d.jL + P::BFL * k];
    }

    for (int c = 0; c < a.C; ++c) {
        if (c + 1 < a.C) {
            load_s(s_nxt, c + 1);
            if (MODE == ROW_INV) load_k(k_nxt, c + 1);
        }
        cf v[R0], u[RL];
        if (MODE != ROW_INV) {
            if (act0) {
#pragma unroll
                for (int m = 0; m < R0; ++m) v[m] = cmul(s_cur[m], xv[m]);
            } else {
#pragma unroll
                for (int m = 0; m < R0; ++m) v[m] = make_float2(0.f, 0.f);
            }
            E::forward(v, u, tw, d, smem, (MODE == ROW_FWD) ? (c & 1) : 0);
        }
        if (MODE == ROW_FUSED) {
            if (actL) {
                if (use_z) {
                    const cf* zrow = a.z + (k_base - d.jL) + c * k_stride;
#pragma unroll
                    for (int k = 0; k < RL; ++k) {
                        u[k] = cscale(u[k], m2v[k]);
                        if (zi[k] >= 0) {
                            const cf q = zrow[zi[k]];
                            u[k] = make_float2(u[k].x - q.x, u[k].y - q.y);
                        }
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < RL; ++k) u[k] = cscale(u[k], m2v[k]);
                }
            }
        } else if (MODE == ROW_FWD) {
            if (actL) {
#pragma unroll
                for (int k = 0; k < RL; ++k) a.W[k_base + c * k_stride + P::BFL * k] = u[k];
            }
        } else {  // ROW_INV
#pragma unroll
            for (int k = 0; k < RL; ++k) u[k] = k_cur[k];
        }
        if (MODE != ROW_FWD) {
            E::inverse(u, v, tw, d, smem, (MODE == ROW_INV) ? (c & 1) : 0);
            if (act0) {
#pragma unroll
                for (int m = 0; m < R0; ++m) {
                    const cf sv = s_cur[m];
                    // acc += conj(s) * v
                    acc[m].x = fmaf(sv.x, v[m].x, fmaf(sv.y, v[m].y, acc[m].x));
                    acc[m].y = fmaf(sv.x, v[m].y, fmaf(-sv.y, v[m].x, acc[m].y));
                }
            }
        }
#pragma unroll
        for (int m = 0; m < R0; ++m) s_cur[m] = s_nxt[m];
#pragma unroll
        for (int k = 0; k < RL; ++k) k_cur[k] = k_nxt[k];
    }
    if (MODE != ROW_FWD) {
        if (act0) {
            if (MODE == ROW_INV) {
#pragma unroll
                for (int m = 0; m < R0; ++m) xv[m] = load_image(a.x, x_off + d.j0 + P::BF0 * m, a.x_planar, b0, a.plane);
            }
#pragma unroll
            for (int m = 0; m < R0; ++m) {
                const cf av = acc[m];
                store_image(a.out, x_off + d.j0 + P::BF0 * m,
                            make_float2(fmaf(-a.eta, av.x, xv[m].x), fmaf(-a.eta, av.y, xv[m].y)), a.out_planar, b0, a.plane);
            }
        }
    }
}

// --------------------------------------------------------------------------------------------
// COL kernel: L neighbouring strided lines per block.
// --------------------------------------------------------------------------------------------
template <class P, int L, int MODE>
__global__ void __launch_bounds__(LineFFT<P, true, L>::THREADS)
col_kernel(const ColArgs a) {
    grid_launch_dependents();    // a one-pass row kernel behind this launch may be scheduled early
    using E = LineFFT<P, true, L>;
    constexpr int N = P::N, R0 = P::R0, RL = P::RL;
    extern __shared__ float2 smem[];
    // COL_Z launches ztiles blocks per outer index and lets them stride over the tiles of sampled
    // ranks (their number is only known on the device); the other modes launch one block per tile
    const int tiles = (MODE == COL_Z) ? a.ztiles : (a.es + L - 1) / L;
    const long long o = blockIdx.x / tiles;           // outer index
    int i_base = (int)(blockIdx.x % tiles) * L;
    if (MODE == COL_Z && a.zlist != nullptr) {
        // lines are ranks of sampled positions: blocks beyond the sampled count leave at once
        const long long bt0 = (o / ((long long)a.C * a.T)) * a.T + (o % a.T);
        if (i_base >= a.zcount[bt0]) return;
    }
    const typename E::Ids d = E::ids(threadIdx.x);
    typename E::Tw tw;
    E::make_tw(d, tw);

    // COL mode: every stage sees the same line index l = tid % L
    int i = i_base + d.l0;
    const bool line_ok = i < a.es;
    const bool act0 = d.a0 && line_ok, actL = d.aL && line_ok;
    const long long base = o * (long long)N * a.es + i;

    cf v[R0], u[RL];

    if constexpr (MODE == COL_Z) {
      // Without a rank map from an earlier launch (a.zlist == null; rank 2 with at most
      // COLZ_SELF_MAX phase-encode positions) the block ranks the sampled positions of its mask
      // row itself: it lists the source positions sh(q) of the sampled raw k indices q in the
      // order of q -- the order in which the one-pass row kernel counts them.
      __shared__ int s_list[COLZ_SELF_MAX];
      __shared__ unsigned s_bal[COLZ_SELF_MAX / 32];
      const bool self_ranks = a.zlist == nullptr;
      int self_cnt = 0;
      if (self_ranks) {
          const long long bt0 = (o / ((long long)a.C * a.T)) * a.T + (o % a.T);
          const float* mk = a.mask + bt0 * a.es;
          const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
          const int nchunks = (a.es + 31) / 32;
          // every warp marks the sampled entries of its chunks of 32 raw indices ...
          for (int c = warp; c < nchunks; c += nwarps) {
              const int q = c * 32 + lane;
              const bool on = (q < a.es) && (mk[shift_half(q, a.es)] != 0.f);
              const unsigned bal = __ballot_sync(0xffffffffu, on);
              if (lane == 0) s_bal[c] = bal;
          }
          __syncthreads();
          // ... then numbers them behind the entries of the chunks before
          for (int c = warp; c < nchunks; c += nwarps) {
              int before = 0;
              for (int e = 0; e < c; ++e) before += __popc(s_bal[e]);
              const unsigned bal = s_bal[c];
              const int q = c * 32 + lane;
              if ((bal >> lane) & 1u) s_list[before + __popc(bal & ((1u << lane) - 1u))] = shift_half(q, a.es);
          }
          for (int e = 0; e < nchunks; ++e) self_cnt += __popc(s_bal[e]);
          __syncthreads();
          if (i_base >= self_cnt) return;
      }
      for (;; i_base += tiles * L, i += tiles * L) {
        // Lines are the sampled phase-encode positions of this unit's (b,t), by rank r.
        // z[r] = (g/sqrt(N_ro N_pe)) (-1)^{n_ro} (-1)^{p} M[p] * Rraw^H( (-1)^{k_ro} y[.., p] ),  p = zlist[r]
        const int t = (int)(o % a.T);
        const int b = (int)(o / ((long long)a.C * a.T));
        const long long bt = (long long)b * a.T + t;
        const long long pe = a.es;
        const int cnt = self_ranks ? self_cnt : a.zcount[bt];
        if (i_base >= cnt) return;                      // no tile of sampled ranks left for this block
        const bool ok = i < cnt;
        int p = 0, psign = 0; float mv = 0.f;
        if (ok) {
            p = self_ranks ? s_list[i] : a.zlist[bt * pe + i];
            mv = a.mask[bt * pe + p];
            psign = (a.rank == 2) ? (p & 1) : ((p / a.n2 + p % a.n2) & 1);
        }
        if (d.aL && ok) {
#pragma unroll
            for (int k = 0; k < RL; ++k) {
                const int kk = d.jL + P::BFL * k;
                const cf yv = a.y[o * (long long)N * pe + (long long)kk * pe + p];
                u[k] = (kk & 1) ? make_float2(-yv.x, -yv.y) : yv;
            }
        }
        E::inverse(u, v, tw, d, smem);
        if (d.a0 && ok) {
            const float f = (psign ? -a.scale : a.scale) * mv;
#pragma unroll
            for (int m = 0; m < R0; ++m) {
                const int n = d.j0 + P::BF0 * m;
                const float ff = (n & 1) ? -f : f;
                a.z[o * (long long)N * pe + (long long)n * pe + i] = cscale(v[m], ff);
            }
        }
        __syncthreads();                                // exchange buffer is reused by the next tile
      }
    }

    if (MODE == COL_INV) {
        if (actL) {
#pragma unroll
            for (int k = 0; k < RL; ++k) u[k] = a.W[base + (long long)(d.jL + P::BFL * k) * a.es];
        }
    } else {
        if (act0) {
#pragma unroll
            for (int m = 0; m < R0; ++m) v[m] = a.W[base + (long long)(d.j0 + P::BF0 * m) * a.es];
        } else {
#pragma unroll
            for (int m = 0; m < R0; ++m) v[m] = make_float2(0.f, 0.f);
        }
        E::forward(v, u, tw, d, smem);
    }

    if (MODE == COL_FWD) {
        if (actL) {
#pragma unroll
            for (int k = 0; k < RL; ++k) a.W[base + (long long)(d.jL + P::BFL * k) * a.es] = u[k];
        }
        return;
    }

    if (MODE == COL_MID_SEP) {
        // W chunk (unit, G, n1, n2), axis n1, es = n2.  o = unit*G + gi
        if (actL) {
            const long long unit = o / a.G;
            const int gi = (int)(o % a.G);
            const int t = (int)(unit % a.T);
            const int b = (int)(unit / ((long long)a.C * a.T));
            const long long pe = (long long)a.n1 * a.n2;
            const float* mk = a.mask + ((long long)b * a.T + t) * pe + shift_half(i, a.n2);
            const cf* zz = a.zin ? a.zin + (unit * a.n0 + a.i0_start + gi) * pe : nullptr;
            const int* zi = a.zidx + ((long long)b * a.T + t) * pe + i;
#pragma unroll
            for (int k = 0; k < RL; ++k) {
                const long long kk = (long long)(d.jL + P::BFL * k) * a.n2;
                const float mv = mk[(long long)shift_half(d.jL + P::BFL * k, N) * a.n2];
                const float w = mv * mv * a.scale2;
                u[k] = cscale(u[k], w);
                if (zz && mv != 0.f) {
                    const cf q = zz[zi[kk]];
                    u[k] = make_float2(u[k].x - q.x, u[k].y - q.y);
                }
            }
        }
    } else if (MODE == COL_MID_FULL) {
        // W (unit, V); the transformed axis is the readout axis (n1 for rank 2, n0 for rank 3);
        // mask and y are read at the half-shifted k-space position on every transformed axis.
        if (actL) {
            const long long unit = o;
            const int t = (int)(unit % a.T);
            const int b = (int)(unit / ((long long)a.C * a.T));
            const long long V = (long long)a.n0 * a.n1 * a.n2;
            const float* mk = a.mask + ((long long)b * a.T + t) * V;
            const cf* yy = a.y ? a.y + unit * V : nullptr;
#pragma unroll
            for (int k = 0; k < RL; ++k) {
                const int kk = d.jL + P::BFL * k;
                long long ps; int par;
                if (a.rank == 2) {
                    const int s1 = shift_half(kk, a.n1), s2 = shift_half(i, a.n2);
                    ps = (long long)s1 * a.n2 + s2; par = (s1 + s2) & 1;
                } else {
                    const int i1 = i / a.n2, i2 = i % a.n2;
                    const int s0 = shift_half(kk, a.n0), s1 = shift_half(i1, a.n1), s2 = shift_half(i2, a.n2);
                    ps = ((long long)s0 * a.n1 + s1) * a.n2 + s2; par = (s0 + s1 + s2) & 1;
                }
                const float mv = mk[ps];
                const float w = mv * mv * a.scale2;
                if (yy) {
                    // measurements at unsampled positions are not read (they may hold anything)
                    const cf q = (mv != 0.f) ? yy[ps] : make_float2(0.f, 0.f);
                    const float f = (par ? -a.scale : a.scale) * mv;
                    u[k] = make_float2(fmaf(w, u[k].x, -f * q.x), fmaf(w, u[k].y, -f * q.y));
                } else {
                    u[k] = cscale(u[k], w);
                }
            }
        }
    }

    if (MODE == COL_GRADY) {
        // Last axis of the forward operator A = Omega F S (Eq. 1) on W (already transformed along the other
        // axes): out[p] = scale (-1)^{|p|} M[p] Fraw(.)[k] at the centred position p = sh(k) of every axis;
        // `scale` carries the caller's factor (eta for the gradient with respect to y), g and 1/sqrt(Ntot).
        if (actL) {
            const long long unit = o;
            const int t = (int)(unit % a.T);
            const int b = (int)(unit / ((long long)a.C * a.T));
            const long long V = (long long)a.n0 * a.n1 * a.n2;
            const long long bt = (long long)b * a.T + t;
            cf* dst = a.ky_out + unit * V;
#pragma unroll
            for (int k = 0; k < RL; ++k) {
                const int kk = d.jL + P::BFL * k;
                long long ps; int par;
                if (a.rank == 2) {
                    const int s1 = shift_half(kk, a.n1), s2 = shift_half(i, a.n2);
                    ps = (long long)s1 * a.n2 + s2; par = (s1 + s2) & 1;
                } else {
                    const int i1 = i / a.n2, i2 = i % a.n2;
                    const int s0 = shift_half(kk, a.n0), s1 = shift_half(i1, a.n1), s2 = shift_half(i2, a.n2);
                    ps = ((long long)s0 * a.n1 + s1) * a.n2 + s2; par = (s0 + s1 + s2) & 1;
                }
                const float mv = a.mask_pe ? a.mask[bt * a.mask_pe + ps % a.mask_pe] : a.mask[bt * V + ps];
                const float f = (par ? -a.scale : a.scale) * mv;
                dst[ps] = cscale(u[k], f);
            }
        }
        return;
    }

    E::inverse(u, v, tw, d, smem);
    if (act0) {
#pragma unroll
        for (int m = 0; m < R0; ++m) a.W[base + (long long)(d.j0 + P::BF0 * m) * a.es] = v[m];
    }
}

}  // namespace gleam
