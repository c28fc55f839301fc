// Warp-resident variant of the ROW kernels (contiguous axis) for plans whose stages need at most
// 32 butterflies per line: every warp owns LW whole lines, so the stage hand-over through shared
// memory needs only __syncwarp(), warps never wait for one another, and the next coil's operands
// stream into shared memory with cp.async while the current coil is transformed.
//
// Same arithmetic as row_kernel (dc_kernels.cuh):
//   ROW_FUSED : out = x - eta * sum_c conj(S_c) Fraw^H ( m2 .* Fraw(S_c x) - z_c )
//   ROW_FWD   : W_c = Fraw(S_c x)                       (k-distribution order = natural order)
//   ROW_INV   : out = x - eta * sum_c conj(S_c) Fraw^H W_c
#pragma once
#include "dc_kernels.cuh"

namespace gleam {

constexpr int pow2_ceil(int v) { int p = 1; while (p < v) p *= 2; return p; }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int NKEEP> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(NKEEP) : "memory");
}

template <class P, int MODE, bool HAS_Z = false>
struct WarpLine {
    static constexpr int N = P::N, R0 = P::R0, RL = P::RL, S = P::S;
    static constexpr int BFMAX = cmax(P::BF0, P::BFL);
    static constexpr bool ELIGIBLE = (S <= 2) && (BFMAX <= 32) && (N % 2 == 0);
    static constexpr int TPL = pow2_ceil(BFMAX);          // lanes per line
    static constexpr int LW = 32 / TPL;                   // lines per warp
    static constexpr int EXL = (S == 2) ? P::SM_A : 0;    // exchange elements per line
    // per-warp shared memory, in float2 units: S[2], K[2] (z or W; not in ROW_FWD), x (not in
    // ROW_INV), exchange, m2 (ROW_FUSED; floats, N/2 float2 per line)
    // K stage: a whole line of the workspace (ROW_INV), or up to KCAP sampled z entries per line
    // (ROW_FUSED with z; lines with more sampled positions read z straight from global memory).
    static constexpr int TILE = LW * N;
    static constexpr int KCAP = (MODE == ROW_INV) ? N : (((N + 3) / 4 + 1) / 2 * 2);
    // ROW_FUSED with z: slot KCAP of every line's stage holds zero; unsampled entries point at it,
    // which keeps the k-space update free of branches
    static constexpr int KSTRIDE = (MODE == ROW_INV) ? KCAP : KCAP + 2;
    static constexpr int KTILE = LW * KSTRIDE;
    static constexpr bool HAS_K = (MODE == ROW_INV) || (MODE == ROW_FUSED && HAS_Z);
    static constexpr bool HAS_X = (MODE == ROW_FUSED);   // ROW_FWD and ROW_INV keep x in registers
    static constexpr bool HAS_M = (MODE == ROW_FUSED), HAS_I = (MODE == ROW_FUSED && HAS_Z);
    static constexpr int OFF_S = 0, OFF_K = 2 * TILE, OFF_X = OFF_K + (HAS_K ? 2 * KTILE : 0),
                         OFF_EX = OFF_X + (HAS_X ? TILE : 0), OFF_M2 = OFF_EX + LW * EXL + (LW * EXL) % 2;
    static constexpr int OFF_IDX = OFF_M2 + (HAS_M ? TILE / 2 : 0);     // ranks of the raw k indices (ints)
    static constexpr int WARP_ELEMS = OFF_IDX + (HAS_I ? TILE / 2 : 0) + 2;
    static constexpr int WARP_ELEMS_ALIGNED = (WARP_ELEMS + 1) / 2 * 2;   // keep 16-byte alignment per warp
};

template <int MODE, bool HAS_Z> __device__ __forceinline__ constexpr bool use_z_slots() { return MODE == ROW_FUSED && HAS_Z; }

template <class P, int WARPS, int MODE, bool HAS_Z>
__global__ void __launch_bounds__(WARPS * 32)
warpline_kernel(const RowArgs a) {
    grid_dependency_wait();
    grid_launch_dependents();
    using WL = WarpLine<P, MODE, HAS_Z>;
    constexpr int KCAP = WL::KCAP, KTILE = WL::KTILE, KSTRIDE = WL::KSTRIDE;
    constexpr int N = P::N, R0 = P::R0, RL = P::RL, TPL = WL::TPL, LW = WL::LW, TILE = WL::TILE;
    extern __shared__ __align__(16) float2 smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    cf* wsm = smem + (size_t)warp * WL::WARP_ELEMS_ALIGNED;
    cf* sS = wsm + WL::OFF_S;
    cf* sK = wsm + WL::OFF_K;
    cf* sX = wsm + WL::OFF_X;
    cf* sE = wsm + WL::OFF_EX;
    float* sM = reinterpret_cast<float*>(wsm + WL::OFF_M2);
    int* sI = reinterpret_cast<int*>(wsm + WL::OFF_IDX);

    const int l = lane / TPL, j = lane % TPL;
    const bool a0 = j < P::BF0, aL = j < P::BFL;

    cf tw0[R0];
    if (P::S == 2) {
#pragma unroll
        for (int k = 0; k < R0; ++k) tw0[k] = unit_root_fwd<N>((j * k) % N);
    }

    if (use_z_slots<MODE, HAS_Z>()) {
        for (int i = lane; i < 2 * LW; i += 32) sK[(i / LW) * KTILE + (i % LW) * KSTRIDE + KCAP] = make_float2(0.f, 0.f);
        __syncwarp();
    }
    const long long ngroups = (a.nrows + LW - 1) / LW;
    const long long wstride = (long long)gridDim.x * WARPS;
    constexpr bool use_z = (MODE == ROW_FUSED) && HAS_Z;
    constexpr bool use_k = (MODE == ROW_INV) || use_z;

    for (long long g = (long long)blockIdx.x * WARPS + warp; g < ngroups; g += wstride) {
        // ---- element offsets of this lane's line; other lines' offsets come by shuffle ----
        const long long row = g * LW + l;
        const bool row_ok = row < a.nrows;
        const unsigned rowu = row_ok ? (unsigned)row : 0u;       // host side guarantees nrows < 2^31
        const unsigned bt = rowu / (unsigned)a.rpb;
        const int ri = (int)(rowu - bt * (unsigned)a.rpb);
        const int b = (int)(bt / (unsigned)a.T), t = (int)(bt - (unsigned)b * (unsigned)a.T);
        const long long x_off = ((long long)bt * a.RPB + a.row0 + ri) * N;
        const long long s_off = (((long long)(b * a.C) * a.Ts + (a.Ts > 1 ? t : 0)) * a.RPB + a.row0 + ri) * N;
        const long long k_off = (MODE == ROW_FUSED) ? (((long long)(b * a.C) * a.T + t) * a.RPB + a.row0 + ri) * N
                                                    : (((long long)(b * a.C) * a.T + t) * a.rpb + ri) * N;
        const long long s_stride = (long long)a.Ts * a.RPB * N;
        const long long k_stride = (long long)a.T * ((MODE == ROW_FUSED) ? a.RPB : a.rpb) * N;

        // entries of this line's K row to stage: the whole row (ROW_INV) or the number of sampled
        // positions (z; set below, when the mask row is scanned)
        int k_cnt = (MODE == ROW_INV) ? N : 0;

        auto issue_coil = [&](int c, int buf) {
#pragma unroll
            for (int ll = 0; ll < LW; ++ll) {
                const bool ok = __shfl_sync(0xffffffffu, (int)row_ok, ll * TPL) != 0;
                const long long so = __shfl_sync(0xffffffffu, s_off, ll * TPL);
                const long long ko = __shfl_sync(0xffffffffu, k_off, ll * TPL);
                const int kc = __shfl_sync(0xffffffffu, k_cnt, ll * TPL);
                if (!ok) continue;
                const cf* src = a.sens + so + c * s_stride;
                for (int i = lane; i < N / 2; i += 32) cp_async16(sS + buf * TILE + ll * N + 2 * i, src + 2 * i);
                if (use_k && kc <= KCAP) {
                    const cf* ks = ((MODE == ROW_FUSED) ? a.z : a.W) + ko + c * k_stride;
                    for (int i = lane; i < (kc + 1) / 2; i += 32) cp_async16(sK + buf * KTILE + ll * KSTRIDE + 2 * i, ks + 2 * i);
                }
            }
        };

        __syncwarp();   // previous group's shared-memory reads are complete
#pragma unroll
        for (int ll = 0; ll < LW; ++ll) {
            const bool ok = __shfl_sync(0xffffffffu, (int)row_ok, ll * TPL) != 0;
            const long long xo = __shfl_sync(0xffffffffu, x_off, ll * TPL);
            const long long bto = __shfl_sync(0xffffffffu, (long long)bt, ll * TPL);
            if (!ok) continue;
            if (WL::HAS_X) {
                if (!a.x_planar) {
                    for (int i = lane; i < N / 2; i += 32) cp_async16(sX + ll * N + 2 * i, a.x + xo + 2 * i);
                } else {
                    // two-channel layout: the line's real parts and its imaginary parts are two contiguous runs
                    const long long bo = __shfl_sync(0xffffffffu, (long long)b, ll * TPL);
                    const float* xf = reinterpret_cast<const float*>(a.x) + xo + bo * a.plane;
                    float* dst = reinterpret_cast<float*>(sX + ll * N);
                    if (N % 4 == 0) {       // staged as two planes of N floats (16-byte copies), read as pairs below
                        for (int i = lane; i < N / 4; i += 32) { cp_async16(dst + 4 * i, xf + 4 * i); cp_async16(dst + N + 4 * i, xf + a.plane + 4 * i); }
                    } else {
                        for (int i = lane; i < N; i += 32) { dst[2 * i] = xf[i]; dst[2 * i + 1] = xf[a.plane + i]; }
                    }
                }
            }
            if (MODE == ROW_FUSED) {
                // scaled mask^2 in raw k order and, with z, the rank of every sampled k (the order
                // in which the z table was written)
                int cnt = 0;
                for (int k0 = 0; k0 < N; k0 += 32) {
                    const int k = k0 + lane;
                    const float mv = (k < N) ? a.mask[bto * N + shift_half(k, N)] : 0.f;
                    if (k < N) sM[ll * N + k] = mv * mv * (1.0f / N);
                    if (use_z) {
                        const unsigned bal = __ballot_sync(0xffffffffu, mv != 0.f);
                        if (k < N) sI[ll * N + k] = (mv != 0.f) ? cnt + __popc(bal & ((1u << lane) - 1u)) : -1;
                        cnt += __popc(bal);
                    }
                }
                if (use_z && l == ll) k_cnt = cnt;
            }
        }
        issue_coil(0, 0);
        cp_async_commit();

        cf acc[R0];
        cf xreg[R0];     // ROW_FWD / ROW_INV: x fetched once per group and held in registers
        if (!WL::HAS_X && a0 && row_ok) {
#pragma unroll
            for (int m = 0; m < R0; ++m) xreg[m] = load_image(a.x, x_off + j + P::BF0 * m, a.x_planar, b, a.plane);
        }
#pragma unroll
        for (int m = 0; m < R0; ++m)
            acc[m] = (MODE != ROW_FWD && a0 && row_ok) ? coil_sum_start(a.aty, x_off + j + P::BF0 * m) : make_float2(0.f, 0.f);

        for (int c = 0; c < a.C; ++c) {
            const int buf = c & 1;
            if (c + 1 < a.C) issue_coil(c + 1, buf ^ 1);
            cp_async_commit();
            cp_async_wait<1>();          // everything but the newest group (coil c+1) has landed
            __syncwarp();

            const cf* cS = sS + buf * TILE + l * N;
            const cf* cK = sK + buf * KTILE + l * KSTRIDE;
            const cf* gK = use_z ? a.z + k_off + c * k_stride : nullptr;   // this line's compact z row
            const cf* cX = sX + l * N;
            const bool x_planes = WL::HAS_X && a.x_planar && (N % 4 == 0);       // x staged as two planes of floats
            auto x_at = [&](int idx) -> cf {
                if (!x_planes) return cX[idx];
                const float* xf = reinterpret_cast<const float*>(cX);
                return make_float2(xf[idx], xf[N + idx]);
            };
            cf v[R0], u[RL];
            if (MODE != ROW_INV) {
                if (a0) {
#pragma unroll
                    for (int m = 0; m < R0; ++m) v[m] = cmul(cS[j + P::BF0 * m], WL::HAS_X ? x_at(j + P::BF0 * m) : xreg[m]);
                    Dft<R0, -1>::run(v);
                }
                if (P::S == 2) {
                    if (a0) {
#pragma unroll
                        for (int k = 0; k < R0; ++k)
                            sE[l * WL::EXL + k * P::LS1 + j] = (k == 0) ? v[0] : cmul(v[k], tw0[k]);
                    }
                    __syncwarp();
                    if (aL) {
#pragma unroll
                        for (int m = 0; m < RL; ++m) u[m] = sE[l * WL::EXL + j * P::LS1 + m];
                        Dft<RL, -1>::run(u);
                    }
                    __syncwarp();
                } else {
#pragma unroll
                    for (int k = 0; k < RL; ++k) u[k] = v[k % R0];
                }
            }
            if (MODE == ROW_FUSED) {
                if (aL) {
                    const float* mm = sM + l * N;
                    if (use_z && row_ok && k_cnt <= KCAP) {
                        // staged z: unsampled entries read the zero slot (lanes without a row hold no rank table)
#pragma unroll
                        for (int k = 0; k < RL; ++k) {
                            const float w = mm[j + P::BFL * k];
                            const int r = sI[l * N + j + P::BFL * k];
                            const cf q = cK[(r >= 0) ? r : KCAP];
                            u[k] = make_float2(fmaf(w, u[k].x, -q.x), fmaf(w, u[k].y, -q.y));
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < RL; ++k) {
                            const float w = mm[j + P::BFL * k];
                            u[k] = cscale(u[k], w);
                            if (use_z && row_ok) {      // more sampled entries than the stage holds: from global memory
                                const int r = sI[l * N + j + P::BFL * k];
                                if (r >= 0 && r < N) {
                                    const cf q = gK[r];
                                    u[k] = make_float2(u[k].x - q.x, u[k].y - q.y);
                                }
                            }
                        }
                    }
                }
            } else if (MODE == ROW_FWD) {
                if (aL && row_ok) {
                    cf* dst = a.W + (((long long)(b * a.C + c) * a.T + t) * a.rpb + ri) * N;
#pragma unroll
                    for (int k = 0; k < RL; ++k) dst[j + P::BFL * k] = u[k];
                }
            } else {
                if (aL) {
#pragma unroll
                    for (int k = 0; k < RL; ++k) u[k] = cK[j + P::BFL * k];
                }
            }
            if (MODE != ROW_FWD) {
                if (P::S == 2) {
                    if (aL) {
                        Dft<RL, +1>::run(u);
#pragma unroll
                        for (int m = 0; m < RL; ++m) sE[l * WL::EXL + j * P::LS1 + m] = u[m];
                    }
                    __syncwarp();
                    if (a0) {
#pragma unroll
                        for (int k = 0; k < R0; ++k) {
                            const cf r = sE[l * WL::EXL + k * P::LS1 + j];
                            v[k] = (k == 0) ? r : cmulc(r, tw0[k]);
                        }
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < R0; ++k) v[k] = u[k % RL];
                }
                if (a0) {
                    Dft<R0, +1>::run(v);
#pragma unroll
                    for (int m = 0; m < R0; ++m) {
                        const cf sv = cS[j + P::BF0 * m];
                        acc[m].x = fmaf(sv.x, v[m].x, fmaf(sv.y, v[m].y, acc[m].x));
                        acc[m].y = fmaf(sv.x, v[m].y, fmaf(-sv.y, v[m].x, acc[m].y));
                    }
                }
            }
            __syncwarp();   // all lanes are done with buffer `buf` and the exchange area
        }
        cp_async_wait<0>();
        if (MODE != ROW_FWD) {
            double dsum = 0.0;       // Re<x, out> over this lane's elements (for the caller's inner product)
            if (a0 && row_ok) {
#pragma unroll
                for (int m = 0; m < R0; ++m) {
                    cf xv = xreg[m];
                    if (WL::HAS_X) {
                        const int idx = j + P::BF0 * m;
                        const float* xf = reinterpret_cast<const float*>(sX + l * N);
                        xv = (a.x_planar && (N % 4 == 0)) ? make_float2(xf[idx], xf[N + idx]) : sX[l * N + idx];
                    }
                    const cf av = acc[m];
                    const cf ov = make_float2(fmaf(-a.eta, av.x, xv.x), fmaf(-a.eta, av.y, xv.y));
                    store_image(a.out, x_off + j + P::BF0 * m, ov, a.out_planar, b, a.plane);
                    if (MODE == ROW_FUSED && a.dot_rows != nullptr) dsum += (double)xv.x * ov.x + (double)xv.y * ov.y;
                }
            }
            if (MODE == ROW_FUSED && a.dot_rows != nullptr) {     // the same in every thread
                for (int o = TPL / 2; o > 0; o >>= 1) dsum += __shfl_down_sync(0xffffffffu, dsum, o, TPL);
                if (j == 0 && row_ok) a.dot_rows[row] = dsum;
            }
        }
    }
}

}  // namespace gleam
