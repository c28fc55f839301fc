// One-pass row kernel (ROW_FUSED arithmetic of dc_warpline.cuh) for two-stage plans whose last stage has
// fewer butterflies per line than the first (N = R0 * RL, R0 < RL, RL in {8, 16, 32}): in the plain
// warp-resident form the RL-point butterflies of the last forward stage, the k-space update and the
// first inverse stage keep only R0 of every RL lanes busy (10 of 16 for N = 160).
//
// Here a warp still owns LW = 32 / RL whole lines, and the first / last image-side stages (S x, R0-point
// butterflies, twiddles; conj(S) coil sum) keep their fixed lane = (line, butterfly) assignment, so the
// coil sum stays in registers.  The k-space stages are stateless, so their work units (one RL-point
// butterfly pair with the mask update in between) are numbered across the coils,
//     unit u = coil * UPC + line * R0 + k,       UPC = LW * R0 units per coil,
// and taken 32 at a time, one per lane: every lane is busy whatever R0 is (N = 160, 8 coils: 5 rounds
// of 32 units instead of 8 rounds of 20).  The stage hand-over goes through a small ring of coil slots in
// shared memory: forward image-side stages run ahead just far enough to fill the next round, the
// inverse image-side stage of a coil runs once all its units are through.  The sensitivities are read
// from global memory straight into registers (a round ahead for the forward stage, at the start of the
// stage for the inverse one), which frees the shared memory the ring needs.
#pragma once
#include "dc_warpline.cuh"

namespace gleam {


template <class P, bool HAS_Z, bool SMW = false>
struct WarpFlat {
    static constexpr int N = P::N, R0 = P::R0, RL = P::RL;
    // R0 < RL is where the plain kernel wastes lanes in the RL-point stages; R0 > RL (368 = 23 x 16) also fits: the
    // R0-point butterflies then run on all lanes of the image-side stages and the RL-point ones on numbered units
    static constexpr bool ELIGIBLE = (P::S == 2) && (RL == 8 || RL == 16 || RL == 32) && (R0 != RL) && (N % 2 == 0);
    static constexpr int LW = 32 / RL;                     // lines per warp
    static constexpr int UPC = LW * R0;                    // k-space units per coil
    static constexpr int USTRIDE = RL + 1;                 // odd: a round's 32 units read without bank conflicts
    static constexpr int SLOTS_MIN = (32 + UPC - 1) / UPC + 1;     // coils between first forward and inverse stage
    // a ring whose unit count is a multiple of 16 keeps the bank pattern across the wrap; taken when small
    static constexpr int slots_aligned() {
        for (int s = SLOTS_MIN; s <= SLOTS_MIN + 3; ++s) if ((s * UPC) % 16 == 0) return s;
        return SLOTS_MIN;
    }
    static constexpr int SLOTS = (!SMW && !HAS_Z && slots_aligned() * UPC * USTRIDE * 8 <= 11 * 1024) ? slots_aligned() : SLOTS_MIN;
    static constexpr int ZS = SMW ? SLOTS : SLOTS + 1;     // z rows are requested one forward stage ahead (SMW: in their own stage)
    static constexpr int KCAP = ((N + 3) / 4 + 1) / 2 * 2; // staged z entries per line (more: read from global memory)
    static constexpr int KSTRIDE = KCAP + 2;               // entry KCAP holds zero (unsampled positions point at it)
    static constexpr int KTILE = LW * KSTRIDE;
    static constexpr int MS = N + ((LW > 1 && N % 32 == 0) ? 16 : 0);   // mask row stride (floats): lines on different banks
    // shared memory of the warp, in float2 units
    static constexpr int OFF_X = 0, OFF_E = LW * N, OFF_M2 = OFF_E + SLOTS * UPC * USTRIDE + (SLOTS * UPC * USTRIDE) % 2;
    // mask weights: one float per raw k (no z), or one per sampled rank next to 16-bit ranks of every raw k (with z)
    static constexpr int OFF_IDX = OFF_M2 + ((HAS_Z ? LW * KSTRIDE : LW * MS) + 3) / 4 * 2;
    static constexpr int OFF_K = OFF_IDX + (HAS_Z ? (LW * N + 7) / 8 * 2 : 0);
    static constexpr int OFF_CNT = OFF_K + (HAS_Z ? ZS * KTILE : 0);
    // per line: element offset of its z row (64-bit), sampled count, mask row index
    static constexpr int ELEMS = (OFF_CNT + 2 * LW + 1) / 2 * 2;
    static constexpr size_t WARP_BYTES = sizeof(cf) * ELEMS;      // per warp of the block
};

// SMW = false: one warp per block, blocks stride over the line groups.
// SMW = true (one round, one block per SM, the host sizes the grid): a block of nwhole + 4 nsplit warps.
// A warp's run time grows with the number of warps on its scheduler (the schedulers favour the oldest warp, and
// the last one to finish sets the time), so 4 k + 1 single-warp blocks per SM leave one scheduler with k + 1
// warps and the others waiting for it.  Here the first nwhole warps of the block take one group each, and every
// further set of four warps (one per scheduler) shares ONE more group, a quarter of the coils each; the partial
// coil sums are added in warp order through shared memory.  A quarter of the extra work lands on every scheduler.
// One block per SM also keeps a dependent launch from moving in next to the running one warp by warp, which
// would fill the schedulers unevenly.
// HAS_ATY: the coil sum is kept as aty - sum, starting from the given A^H y image as loaded (no instruction depends on
// the load before the first inverse stage, so its latency is hidden even when a warp has a single group; the coil
// terms are subtracted and the update adds eta times the result: the same bits as sum - aty, since rounding is
// symmetric in the sign).  Normal-equations form of the step; never together
// with z).  A template parameter, not a run-time test of a.aty: with the test in the code the plain call measured
// 11 % slower (17.7 against 16.0 us), although it never takes that branch.
template <class P, bool HAS_Z, bool SMW, bool HAS_ATY>
__global__ void __launch_bounds__(SMW ? 512 : 32, SMW ? 1 : (P::R0 > 16 ? 8 : P::RL == 32 ? 12 : 16))
warpflat_kernel(const RowArgs a, const int nwhole) {
    grid_dependency_wait();
    grid_launch_dependents();
    using WF = WarpFlat<P, HAS_Z, SMW>;
    constexpr int N = P::N, R0 = P::R0, RL = P::RL, LW = WF::LW, UPC = WF::UPC, US = WF::USTRIDE, SLOTS = WF::SLOTS;
    constexpr int KCAP = WF::KCAP, KSTRIDE = WF::KSTRIDE, KTILE = WF::KTILE, ZS = WF::ZS, MS = WF::MS;
    extern __shared__ __align__(16) float2 smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    cf* wsm = smem + warp * WF::ELEMS;
    cf* sX = wsm + WF::OFF_X;
    cf* sE = wsm + WF::OFF_E;
    float* sM = reinterpret_cast<float*>(wsm + WF::OFF_M2);
    short* sI = reinterpret_cast<short*>(wsm + WF::OFF_IDX);
    cf* sK = wsm + WF::OFF_K;
    long long* sKo = reinterpret_cast<long long*>(wsm + WF::OFF_CNT);      // per line: offset of the z row of coil cbase
    int* sC = reinterpret_cast<int*>(wsm + WF::OFF_CNT + LW);              // per line: sampled entries, -1 for a line past the end
    unsigned* sBt = reinterpret_cast<unsigned*>(sC + LW);                   // per line: mask row
    const bool split = SMW && warp >= nwhole;                      // one of four warps that share a group
    const int set = split ? (warp - nwhole) >> 2 : 0, q = split ? (warp - nwhole) & 3 : 0;
    const int cbase = split ? q * a.C / 4 : 0;                     // first coil and number of coils of this warp
    const int nc = split ? (q + 1) * a.C / 4 - cbase : a.C;

    const int l = lane / RL, j = lane % RL;                 // image-side identity: line of the warp, butterfly

    if (HAS_Z) {
        for (int i = lane; i < ZS * LW; i += 32) sK[(i / LW) * KTILE + (i % LW) * KSTRIDE + KCAP] = make_float2(0.f, 0.f);
        if (lane < LW) sM[lane * KSTRIDE + KCAP] = 0.f;
        __syncwarp();
    }
    // inter-stage twiddles exp(-2 pi i j k / N) of this lane (fetching them again before the image-side stages of
    // every round, to free registers for the k-space round, was measured slower: 18.7 against 16.4 us per call)
    cf tw0[R0];
#pragma unroll
    for (int k = 0; k < R0; ++k) tw0[k] = unit_root_fwd<N>((j * k) % N);
    const long long ngroups = (a.nrows + LW - 1) / LW;
    const int total = UPC * nc, rounds = (total + 31) / 32;
    const long long g_first = !SMW ? (long long)blockIdx.x
                            : split ? (long long)(nwhole + set) * gridDim.x + blockIdx.x : (long long)warp * gridDim.x + blockIdx.x;
    const long long g_step = !SMW ? (long long)gridDim.x : ngroups;              // SMW: a single round

    for (long long g = g_first; g < ngroups; g += g_step) {
        const long long row = g * LW + l;
        const bool row_ok = row < a.nrows;
        const unsigned rowu = row_ok ? (unsigned)row : 0u;       // host side guarantees nrows < 2^31
        const unsigned bt = rowu / (unsigned)a.rpb;
        const int ri = (int)(rowu - bt * (unsigned)a.rpb);
        const int b = (int)(bt / (unsigned)a.T), t = (int)(bt - (unsigned)b * (unsigned)a.T);
        const long long x_off = ((long long)bt * a.RPB + a.row0 + ri) * N;
        // coil indices below are relative to cbase
        const long long s_off = (((long long)(b * a.C + cbase) * a.Ts + (a.Ts > 1 ? t : 0)) * a.RPB + a.row0 + ri) * N;
        const long long k_off = (((long long)(b * a.C + cbase) * a.T + t) * a.RPB + a.row0 + ri) * N;
        const long long s_stride = (long long)a.Ts * a.RPB * N;
        const long long k_stride = (long long)a.T * a.RPB * N;
        const cf* sp = a.sens + s_off + j;                       // this lane's sensitivities of coil 0

        __syncwarp();   // the previous group's shared-memory reads are complete
        // ---- x rows, scaled mask^2 in raw k order and (with z) the rank of every sampled k ----
#pragma unroll
        for (int ll = 0; ll < LW; ++ll) {
            const bool ok = __shfl_sync(0xffffffffu, (int)row_ok, ll * RL) != 0;
            const long long xo = __shfl_sync(0xffffffffu, x_off, ll * RL);
            const long long bto = __shfl_sync(0xffffffffu, (long long)bt, ll * RL);
            if (!ok) { if (lane == 0) sC[ll] = -1; continue; }
            if (!a.x_planar) {
                for (int i = lane; i < N / 2; i += 32) cp_async16(sX + ll * N + 2 * i, a.x + xo + 2 * i);
            } else {
                const long long bo = __shfl_sync(0xffffffffu, (long long)b, ll * RL);
                const float* xf = reinterpret_cast<const float*>(a.x) + xo + bo * a.plane;
                float* dst = reinterpret_cast<float*>(sX + ll * N);
                if (N % 4 == 0) {       // staged as two planes of N floats (16-byte copies), read as pairs below
                    for (int i = lane; i < N / 4; i += 32) { cp_async16(dst + 4 * i, xf + 4 * i); cp_async16(dst + N + 4 * i, xf + a.plane + 4 * i); }
                } else {
                    for (int i = lane; i < N; i += 32) { dst[2 * i] = xf[i]; dst[2 * i + 1] = xf[a.plane + i]; }
                }
            }
            int cnt = 0;
            for (int k0 = 0; k0 < N; k0 += 32) {
                const int k = k0 + lane;
                const float mv = (k < N) ? a.mask[bto * N + shift_half(k, N)] : 0.f;
                if (!HAS_Z) {
                    if (k < N) sM[ll * MS + k] = mv * mv * (1.0f / N);
                } else {
                    const unsigned bal = __ballot_sync(0xffffffffu, mv != 0.f);
                    const int r = cnt + __popc(bal & ((1u << lane) - 1u));
                    if (k < N) sI[ll * N + k] = (short)((mv != 0.f) ? r : -1);
                    if (mv != 0.f && r < KCAP) sM[ll * KSTRIDE + r] = mv * mv * (1.0f / N);
                    cnt += __popc(bal);
                }
            }
            if (lane == 0) sC[ll] = cnt;
            if (HAS_Z && lane == ll * RL) { sKo[ll] = k_off; sBt[ll] = bt; }
        }
        __syncwarp();
        // z row of coil c for every line of the warp -> slot c % ZS
        auto issue_z = [&](int c) {
#pragma unroll
            for (int ll = 0; ll < LW; ++ll) {
                const long long ko = sKo[ll];
                const int kc = sC[ll];
                if (kc <= 0 || kc > KCAP) continue;
                const cf* ks = a.z + ko + c * k_stride;
                for (int i = lane; i < (kc + 1) / 2; i += 32) cp_async16(sK + (c % ZS) * KTILE + ll * KSTRIDE + 2 * i, ks + 2 * i);
            }
        };
        constexpr int ZAHEAD = SMW ? 0 : 1;      // forward stages between the request for a z row and the stage of its coil
        if (HAS_Z && ZAHEAD) issue_z(0);
        cp_async_commit();

        const bool x_planes = a.x_planar && (N % 4 == 0);          // x staged as two planes of floats
        const cf* cX = sX + l * N;
        auto x_at = [&](int idx) -> cf {
            if (!x_planes) return cX[idx];
            const float* xf = reinterpret_cast<const float*>(cX);
            return make_float2(xf[idx], xf[N + idx]);
        };
        auto load_sens = [&](cf (&dst)[R0], int c) {
            const cf* p = sp + c * s_stride;
#pragma unroll
            for (int m = 0; m < R0; ++m) dst[m] = row_ok ? __ldg(p + RL * m) : make_float2(0.f, 0.f);
        };

        cf acc[R0];
#pragma unroll
        for (int m = 0; m < R0; ++m) acc[m] = (HAS_ATY && row_ok && q == 0) ? a.aty[x_off + j + RL * m] : make_float2(0.f, 0.f);
        cf sf[R0];                       // sensitivities of the next forward image-side stage
        if (nc > 0) load_sens(sf, 0);
        int af = 0, ai = 0;              // next coil of the forward / of the inverse image-side stage

        for (int br = 0; br < rounds; ++br) {
            const int upto = min(32 * (br + 1), total);
            const int need = (upto + UPC - 1) / UPC;                     // coils this round draws units from
            const int done = (br == rounds - 1) ? nc : upto / UPC;       // coils complete after this round
            // ---- forward image-side stage: S x, R0-point butterflies, twiddles, into the ring ----
            while (af < need) {
                if (HAS_Z) { if (af + ZAHEAD < nc) issue_z(af + ZAHEAD); cp_async_commit(); }
                if (af == 0) { cp_async_wait<HAS_Z ? 1 : 0>(); __syncwarp(); }      // x (and z of coil 0) have landed
                cf v[R0];
#pragma unroll
                for (int m = 0; m < R0; ++m) v[m] = cmul(sf[m], x_at(j + RL * m));
                if (af + 1 < nc) load_sens(sf, af + 1);
                Dft<R0, -1>::run(v);
                cf* e = sE + ((af % SLOTS) * UPC + l * R0) * US + j;
#pragma unroll
                for (int k = 0; k < R0; ++k) e[k * US] = (k == 0) ? v[0] : cmul(v[k], tw0[k]);
                ++af;
            }
            if (HAS_Z) cp_async_wait<ZAHEAD>();  // everything but a request for the next coil's z is there
            __syncwarp();
            // ---- k-space round: units 32 br .. 32 br + 31, one per lane ----
            {
                const int u0 = 32 * br + lane;
                const bool live = u0 < total;
                const int uu = live ? u0 : total - 1;
                const int c = uu / UPC, w = uu - c * UPC;
                const int bl = w / R0, jb = w - bl * R0;
                cf* e = sE + ((c % SLOTS) * UPC + w) * US;
                cf u[RL];
#pragma unroll
                for (int m = 0; m < RL; ++m) u[m] = e[m];
                Dft<RL, -1>::run(u);
                if (!HAS_Z) {
                    const float* mm = sM + bl * MS + jb;
#pragma unroll
                    for (int k = 0; k < RL; ++k) u[k] = cscale(u[k], mm[R0 * k]);
                } else {
                    const int kc = sC[bl];
                    const short* ri_ = sI + bl * N + jb;
                    if (kc > 0 && kc <= KCAP) {
                        // staged z and weights by rank: unsampled entries read the zero slots
                        const float* mw = sM + bl * KSTRIDE;
                        const cf* zk = sK + (c % ZS) * KTILE + bl * KSTRIDE;
#pragma unroll
                        for (int k = 0; k < RL; ++k) {
                            const int r = ri_[R0 * k];
                            const int rr = (r >= 0) ? r : KCAP;
                            const float wv = mw[rr];
                            const cf q = zk[rr];
                            u[k] = make_float2(fmaf(wv, u[k].x, -q.x), fmaf(wv, u[k].y, -q.y));
                            if (k % 4 == 3) asm volatile("" ::: "memory");     // four entries in flight at a time: registers
                        }
                    } else if (kc > KCAP) {
                        // more sampled entries than the stage holds: weights and z from global memory
                        const float* mrow = a.mask + (long long)sBt[bl] * N;
                        const cf* zrow = a.z + sKo[bl] + c * k_stride;
#pragma unroll
                        for (int k = 0; k < RL; ++k) {
                            const float mv = mrow[shift_half(jb + R0 * k, N)];
                            u[k] = cscale(u[k], mv * mv * (1.0f / N));
                            const int r = ri_[R0 * k];
                            if (r >= 0) {
                                const cf q = zrow[r];
                                u[k] = make_float2(u[k].x - q.x, u[k].y - q.y);
                            }
                            asm volatile("" ::: "memory");      // one entry at a time: this rare path must not cost registers
                        }
                    } else {       // nothing sampled on this line (or no line)
#pragma unroll
                        for (int k = 0; k < RL; ++k) u[k] = make_float2(0.f, 0.f);
                    }
                }
                Dft<RL, +1>::run(u);
                if (live) {
#pragma unroll
                    for (int m = 0; m < RL; ++m) e[m] = u[m];
                }
            }
            __syncwarp();
            // ---- inverse image-side stage of the coils that are complete: twiddles, R0-point butterflies, conj(S) sum ----
            while (ai < done) {
                cf si[R0];
                load_sens(si, ai);
                const cf* e = sE + ((ai % SLOTS) * UPC + l * R0) * US + j;
                cf v[R0];
#pragma unroll
                for (int k = 0; k < R0; ++k) {
                    const cf r = e[k * US];
                    v[k] = (k == 0) ? r : cmulc(r, tw0[k]);
                }
                Dft<R0, +1>::run(v);
#pragma unroll
                for (int m = 0; m < R0; ++m) {
                    if (HAS_ATY) {      // acc = aty - sum
                        acc[m].x = fmaf(-si[m].x, v[m].x, fmaf(-si[m].y, v[m].y, acc[m].x));
                        acc[m].y = fmaf(-si[m].x, v[m].y, fmaf(si[m].y, v[m].x, acc[m].y));
                    } else {
                        acc[m].x = fmaf(si[m].x, v[m].x, fmaf(si[m].y, v[m].y, acc[m].x));
                        acc[m].y = fmaf(si[m].x, v[m].y, fmaf(-si[m].y, v[m].x, acc[m].y));
                    }
                }
                ++ai;
            }
        }
        cp_async_wait<0>();
        __syncwarp();
        if (SMW && split) {
            // partial coil sums of the other three warps are added by the first in warp order (the ring is free by now)
            if (q > 0) {
#pragma unroll
                for (int m = 0; m < R0; ++m) sE[m * 32 + lane] = acc[m];
            }
            // the four warps of this group (every one gets here: same g)
            if (set == 0) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync 2, 128;" ::: "memory");
            if (q > 0) continue;
            for (int w = 1; w < 4; ++w) {
                const cf* o = smem + (nwhole + 4 * set + w) * WF::ELEMS + WF::OFF_E;
#pragma unroll
                for (int m = 0; m < R0; ++m) acc[m] = cadd(acc[m], o[m * 32 + lane]);
            }
        }
        // ---- out = x - eta * sum, and Re<x, out> per row for the caller's inner product ----
        double dsum = 0.0;
        if (row_ok) {
#pragma unroll
            for (int m = 0; m < R0; ++m) {
                const cf xv = x_at(j + RL * m);
                const cf av = acc[m];
                const float se = HAS_ATY ? a.eta : -a.eta;          // HAS_ATY: acc holds aty - sum
                const cf ov = make_float2(fmaf(se, av.x, xv.x), fmaf(se, av.y, xv.y));
                store_image(a.out, x_off + j + RL * m, ov, a.out_planar, b, a.plane);
                if (a.dot_rows != nullptr) dsum += (double)xv.x * ov.x + (double)xv.y * ov.y;
            }
        }
        if (a.dot_rows != nullptr) {     // the same in every thread
            for (int o = RL / 2; o > 0; o >>= 1) dsum += __shfl_down_sync(0xffffffffu, dsum, o, RL);
            if (j == 0 && row_ok) a.dot_rows[row] = dsum;
        }
    }
}

}  // namespace gleam
