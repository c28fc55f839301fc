// Pipelined variant of col_kernel<COL_MID_SEP> (strided-axis transform, mask + residual, inverse,
// in place on the workspace chunk) for two-stage plans.
//
// A block is persistent: it walks over tiles of L neighbouring strided lines and, while it
// transforms one tile, the next one streams from the (L2-resident) workspace into shared memory
// with cp.async.  Three shared-memory buffers rotate between the roles "incoming tile",
// "forward exchange" and "inverse exchange" (the buffer the current tile arrived in, once every
// thread holds its elements in registers).
#pragma once
#include "dc_warpline.cuh"

namespace gleam {

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(d), "l"(gsrc) : "memory");
}

template <class P, int L>
struct ColPipe {
    static constexpr bool ELIGIBLE = (P::S == 2) && (L % 2 == 0);
    static constexpr int BUFSZ = L * cmax(P::BUF, P::N);            // elements per buffer
    static constexpr size_t SMEM_BYTES = sizeof(cf) * (3 * BUFSZ + 2);
    static constexpr int THREADS = LineFFT<P, true, L>::THREADS;
    static constexpr int ZCAP = 384;      // sampled entries per tile whose z values are staged (forward call)
    // resident blocks per SM that shared memory allows (227 KB usable), capped at 3
    static constexpr int MIN_BLOCKS = (3 * SMEM_BYTES <= 227 * 1024) ? 3 : ((2 * SMEM_BYTES <= 227 * 1024) ? 2 : 1);
};

// HAS_Z = true is the forward call: the block keeps, instead of the mask weights, the ranks of its
// k-space entries among the sampled positions and fetches weight and z value by rank.
template <class P, int L, bool HAS_Z>
__global__ void __launch_bounds__(ColPipe<P, L>::THREADS, ColPipe<P, L>::MIN_BLOCKS)
colpipe_mid_sep_kernel(const ColArgs a) {
    using E = LineFFT<P, true, L>;
    using CP = ColPipe<P, L>;
    constexpr int N = P::N, R0 = P::R0, RL = P::RL;
    extern __shared__ __align__(16) float2 smem[];
    cf* buf[3] = {smem, smem + CP::BUFSZ, smem + 2 * CP::BUFSZ};
    const typename E::Ids d = E::ids(threadIdx.x);
    typename E::Tw tw;
    E::make_tw(d, tw);

    // tile counters are 32-bit (the launcher refuses more than 2^31 tiles): no 64-bit divisions
    const unsigned tiles_per_o = (unsigned)((a.es + L - 1) / L);
    const long long pe = (long long)a.n1 * a.n2;

    // Work order: the grid is a whole number of "rows" of tiles_per_o blocks; block b keeps column
    // tile b % tiles_per_o and walks over the outer indices o = b / tiles_per_o, + rows, ...  so the
    // mask weights of its k-space entries stay in registers from one tile to the next.
    const unsigned col_tile = blockIdx.x % tiles_per_o;
    const unsigned rows = gridDim.x / tiles_per_o;            // host launches a multiple of tiles_per_o
    const unsigned nout = (unsigned)a.nouter;

    // stream the tile of outer index o into `dst` in [n][l] layout; chunks of 16 bytes
    // slot ZCAP of s_wt / s_z is a dummy that holds zero: unsampled entries point at it, which keeps
    // the k-space update free of branches
    __shared__ int s_rank[HAS_Z ? CP::ZCAP : 1];        // ranks of the tile's sampled entries (forward call)
    __shared__ float s_wt[HAS_Z ? CP::ZCAP + 1 : 1];    // their scaled squared mask weights
    __shared__ cf s_z[2][HAS_Z ? CP::ZCAP + 1 : 1];     // their z values, double-buffered over tiles
    __shared__ int s_wcnt[CP::THREADS / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int z_total = 0;            // sampled entries of this block's column tile
    bool z_staged = false;      // they fit the staging area

    // z values of the tile of outer index o -> s_z[slot] (asynchronous, 8 bytes each)
    auto issue_z = [&](unsigned o, int slot) {
        const unsigned unit = o / (unsigned)a.G;
        const int gi = (int)(o - unit * (unsigned)a.G);
        const cf* zz = a.zin + ((long long)unit * a.n0 + a.i0_start + gi) * pe;
        for (int e = threadIdx.x; e < z_total; e += CP::THREADS) cp_async8(&s_z[slot][e], zz + s_rank[e]);
    };

    auto issue = [&](unsigned o, cf* dst) {
        const int i_base = (int)col_tile * L;
        const cf* src = a.W + o * (long long)N * a.es + i_base;
        for (int c = threadIdx.x; c < N * (L / 2); c += CP::THREADS) {
            const int n = c / (L / 2), part = c - n * (L / 2);
            if (i_base + 2 * part < a.es) cp_async16(dst + n * L + 2 * part, src + (long long)n * a.es + 2 * part);
        }
    };

    unsigned o = blockIdx.x / tiles_per_o;
    if (o < nout) issue(o, buf[0]);
    cp_async_commit();
    int it = 0;
    long long bt_loaded = -1;
    float mw[RL];       // VJP: mask weights of this thread's k-space entries
    unsigned zp[(RL + 1) / 2];   // forward: positions of this thread's entries in the tile's staged list, two
                                 // 16-bit values per register (ZCAP = the zero dummy slot: unsampled entry)
    for (; o < nout; o += rows, ++it) {
        cf* cur = buf[it % 3];
        cf* nxt = buf[(it + 1) % 3];
        cf* spare = buf[(it + 2) % 3];
        cp_async_wait<0>();
        __syncthreads();          // tile is visible to all; every thread has left the previous tile
        if (o + rows < nout) issue(o + rows, nxt);
        cp_async_commit();

        const int i_base = (int)col_tile * L;
        const int i = i_base + d.l0;
        const bool line_ok = i < a.es;
        const bool act0 = d.a0 && line_ok, actL = d.aL && line_ok;
        const long long base = o * (long long)N * a.es + i;
        // chunk geometry: o = unit * G + gi
        const unsigned unit = o / (unsigned)a.G;
        const int gi = (int)(o - unit * (unsigned)a.G);
        const unsigned bc = unit / (unsigned)a.T;
        const int t = (int)(unit - bc * (unsigned)a.T);
        const int b = (int)(bc / (unsigned)a.C);
        const long long bt = (long long)b * a.T + t;

        cf v[R0], u[RL];
        if (act0) {
#pragma unroll
            for (int m = 0; m < R0; ++m) v[m] = cur[(d.j0 + P::BF0 * m) * L + d.l0];
        } else {
#pragma unroll
            for (int m = 0; m < R0; ++m) v[m] = make_float2(0.f, 0.f);
        }
        if (bt != bt_loaded) {   // per-(b,t) tables of this thread's k-space entries: reloaded only when (b,t) changes
            bt_loaded = bt;
            if (HAS_Z) {
                // Ranks of this thread's entries among the sampled positions.  The sampled entries of
                // the whole tile are then numbered block-wide; their ranks and weights go to shared
                // memory, and every later tile fetches its z values asynchronously, one tile ahead.
                const int* zi = a.zidx + bt * pe + i;
                const float* m2 = a.m2c + bt * pe;
                int zr[RL];
#pragma unroll
                for (int k = 0; k < RL; ++k) zr[k] = actL ? zi[(long long)(d.jL + P::BFL * k) * a.n2] : -1;
                int wc = 0;
#pragma unroll
                for (int k = 0; k < RL; ++k) wc += __popc(__ballot_sync(0xffffffffu, zr[k] >= 0));
                __syncthreads();                       // earlier readers of the tables are done
                if (lane == 0) s_wcnt[warp] = wc;
                __syncthreads();
                int base = 0, total = 0;
                for (int w2 = 0; w2 < CP::THREADS / 32; ++w2) { if (w2 < warp) base += s_wcnt[w2]; total += s_wcnt[w2]; }
                z_total = total;
                z_staged = total <= CP::ZCAP;
                if (z_staged) {
                    if (threadIdx.x == 0) {
                        s_wt[CP::ZCAP] = 0.f;
                        s_z[0][CP::ZCAP] = make_float2(0.f, 0.f);
                        s_z[1][CP::ZCAP] = make_float2(0.f, 0.f);
                    }
#pragma unroll
                    for (int k = 0; k < RL; ++k) {
                        const bool on = zr[k] >= 0;
                        const unsigned bal = __ballot_sync(0xffffffffu, on);
                        int pos = CP::ZCAP;
                        if (on) {
                            pos = base + __popc(bal & ((1u << lane) - 1u));
                            s_rank[pos] = zr[k];
                            s_wt[pos] = m2[zr[k]] * a.scale2;
                        }
                        if (k % 2 == 0) zp[k / 2] = (unsigned)pos;
                        else zp[k / 2] |= (unsigned)pos << 16;
                        base += __popc(bal);
                    }
                    __syncthreads();
                    issue_z(o, it & 1);                // this tile's values were not prefetched
                    cp_async_commit();
                    cp_async_wait<0>();
                    __syncthreads();
                }
            } else if (actL) {
                const float* mk = a.mask + bt * pe + shift_half(i, a.n2);
#pragma unroll
                for (int k = 0; k < RL; ++k) mw[k] = mk[(long long)shift_half(d.jL + P::BFL * k, N) * a.n2];
            }
        }
        if (HAS_Z && z_staged && o + rows < nout) {   // z values of the next tile, one tile ahead
            issue_z(o + rows, (it + 1) & 1);
            cp_async_commit();
        }
        // forward exchange in `spare` (free since the barrier above); every thread has read its
        // elements from `cur` before it passes the barrier inside forward_xy, so `cur` can take
        // the inverse exchange afterwards
        E::forward_xy(v, u, tw, d, spare, spare);
        if (HAS_Z) {
            if (actL && z_staged) {
                const cf* zs = s_z[it & 1];
#pragma unroll
                for (int k = 0; k < RL; ++k) {
                    const int pos = (k % 2 == 0) ? (int)(zp[k / 2] & 0xffffu) : (int)(zp[k / 2] >> 16);
                    const float w = s_wt[pos];
                    const cf q = zs[pos];
                    u[k] = make_float2(fmaf(w, u[k].x, -q.x), fmaf(w, u[k].y, -q.y));
                }
            } else if (actL) {     // more sampled entries than the staging area holds: fetch directly
                const cf* zz = a.zin + ((long long)unit * a.n0 + a.i0_start + gi) * pe;
                const float* m2 = a.m2c + bt * pe;
                const int* zi = a.zidx + bt * pe + i;
#pragma unroll
                for (int k = 0; k < RL; ++k) {
                    const int r = zi[(long long)(d.jL + P::BFL * k) * a.n2];
                    if (r >= 0) {
                        const float w = m2[r] * a.scale2;
                        const cf q = zz[r];
                        u[k] = make_float2(fmaf(w, u[k].x, -q.x), fmaf(w, u[k].y, -q.y));
                    } else {
                        u[k] = make_float2(0.f, 0.f);
                    }
                }
            }
        } else if (actL) {
#pragma unroll
            for (int k = 0; k < RL; ++k) u[k] = cscale(u[k], mw[k] * mw[k] * a.scale2);
        }
        E::inverse_xy(u, v, tw, d, cur, cur);
        if (act0) {
#pragma unroll
            for (int m = 0; m < R0; ++m) a.W[base + (long long)(d.j0 + P::BF0 * m) * a.es] = v[m];
        }
    }
    cp_async_wait<0>();
}

}  // namespace gleam
