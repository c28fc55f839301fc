// Row-tile kernels for the separable 3-D path: a 2-D transform over (ky, kz) split so that every
// pass over the workspace is contiguous in memory.
//
// ky has the two-stage plan N1 = RY * BY (first radix RY, BY = N1 / RY butterflies), kz the
// warp-resident plan PZ.  With ky = j + BY m (m < RY) on the image side and ky = k0 + RY k1 (k1 < BY)
// on the k-space side:
//   pass 1  rowtile_fwd : block (b,t,i0,j) takes the RY rows ky = j + BY m, multiplies by S_c,
//                         transforms each row along kz (one warp per LW rows), then transforms the
//                         RY rows against each other (radix RY, one thread per kz), applies the
//                         ky twiddle w_N1^(j k0) and stores  V[unit][i0][k0][j][kz].
//   pass 2  rowtile_mid : block (unit,i0,k0) reads the BY contiguous rows V[..][k0][0..BY)[kz],
//                         radix-BY transform over j (-> k1), mask^2 / (N1 NZ) and - z at the raw
//                         position (k0 + RY k1, kz), inverse radix BY, stores in place.
//   pass 3  rowtile_inv : mirror of pass 1 with the conjugate-sensitivity coil sum and the update.
// The three passes compute exactly what row_fwd / col_mid_sep / row_inv compute.
#pragma once
#include "size_ops.cuh"

namespace gleam {

struct TileArgs {
    const cf* x; const cf* sens; cf* out;     // image side (pass 1, 3)
    cf* V;                                    // workspace (unit, G, RY, BY, NZ)
    const float* mask;                        // (B,T,N1,NZ) readout-invariant mask (pass 2)
    const cf* zin; const int* zidx;           // compact z table and rank map (pass 2, forward call)
    const float* m2c;                         // squared mask weights by rank (pass 2, forward call)
    const int* zstart;                        // (B,T,33): first rank of each ky-mod-RY group
    float eta, scale2;
    int C, T, Ts, n0, G, i0_start;
    long long nunits;                         // B*C*T
    int x_planar, out_planar; long long plane; // two-real-channel layout of x / out (see RowArgs)
    const cf* aty;                            // A^H y image of the normal-equations form, or null (see RowArgs)
};

template <class PZ, int RY, int BY>
struct RowTile {
    using WL = WarpLine<PZ, ROW_FWD, false>;
    static constexpr int NZ = PZ::N, N1 = RY * BY;
    static constexpr bool ELIGIBLE = WL::ELIGIBLE && (PZ::S == 2) && (RY % WL::LW == 0) && (RY / WL::LW <= 32);
    static constexpr int WARPS = RY / WL::LW;              // one warp per LW of the RY rows
    static constexpr int THREADS = WARPS * 32;
    // shared memory (float2 units): tile T[RY][NZ], then per warp: S[LW*NZ] and the exchange area
    static constexpr int TILE_T = RY * NZ;
    static constexpr int PER_WARP = WL::TILE + WL::LW * WL::EXL + (WL::LW * WL::EXL) % 2;   // S rows (single buffer) + exchange
    static constexpr size_t SMEM_BYTES = sizeof(cf) * (TILE_T + WARPS * PER_WARP + 2);
};

// ---------------------------------------------------------------------------------------------
// pass 1 (INV = false) and pass 3 (INV = true)
// ---------------------------------------------------------------------------------------------
template <class PZ, int RY, int BY, bool INV>
__global__ void __launch_bounds__(RowTile<PZ, RY, BY>::THREADS, INV ? 1 : 2)
rowtile_kernel(const TileArgs a) {
    using RT = RowTile<PZ, RY, BY>;
    using WL = typename RT::WL;
    constexpr int NZ = PZ::N, R0 = PZ::R0, RL = PZ::RL, TPL = WL::TPL, LW = WL::LW, N1 = RY * BY;
    extern __shared__ __align__(16) float2 smem[];
    cf* sT = smem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    cf* wsm = smem + RT::TILE_T + warp * RT::PER_WARP;
    cf* sS = wsm;
    cf* sE = wsm + WL::TILE;

    // block -> (bt, slab gi of the chunk, j)
    const unsigned blk = blockIdx.x;
    const unsigned j_y = blk % BY;
    const unsigned gi = (blk / BY) % (unsigned)a.G;
    const unsigned bt = blk / (BY * (unsigned)a.G);
    const int b = (int)(bt / (unsigned)a.T), t = (int)(bt - (unsigned)b * a.T);
    const int i0 = a.i0_start + (int)gi;

    // this lane's row of the tile and its place in the kz line
    const int l = lane / TPL, jz = lane % TPL;
    const int m_row = warp * LW + l;                         // 0 .. RY-1
    const int ky = (int)j_y + BY * m_row;                    // image-side row
    const bool a0 = jz < PZ::BF0, aL = jz < PZ::BFL;
    const long long row_elems = ((long long)i0 * N1 + ky) * NZ;              // inside one (n0,N1,NZ) volume
    const long long V3 = (long long)a.n0 * N1 * NZ;
    const long long x_off = (long long)bt * V3 + row_elems;
    const long long s_off = ((long long)(b * a.C) * a.Ts + (a.Ts > 1 ? t : 0)) * V3 + row_elems;
    const long long s_stride = (long long)a.Ts * V3;

    cf twz[R0];                                              // kz inter-stage twiddles of this lane
#pragma unroll
    for (int k = 0; k < R0; ++k) twz[k] = unit_root_fwd<NZ>((jz * k) % NZ);

    // S rows of this warp for coil c.  Single buffer: the copy for the next coil is issued as soon
    // as the warp has consumed the current one and lands while the rest of the iteration runs.
    auto issue_s = [&](int c) {
#pragma unroll
        for (int ll = 0; ll < LW; ++ll) {
            const long long so = __shfl_sync(0xffffffffu, s_off, ll * TPL);
            const cf* src = a.sens + so + c * s_stride;
            for (int i = lane; i < NZ / 2; i += 32) cp_async16(sS + ll * NZ + 2 * i, src + 2 * i);
        }
        cp_async_commit();
    };
    // ky twiddles of this block's rows: w_N1^(j k0)
    cf twy[RY];
#pragma unroll
    for (int k0 = 0; k0 < RY; ++k0) twy[k0] = unit_root_fwd<N1>(((int)j_y * k0) % N1);
    auto v_ptr = [&](int c) -> cf* {                         // V[unit][gi][.][j][.] of coil c
        const long long unit = ((long long)(b * a.C + c)) * a.T + t;
        return a.V + (((unit * a.G + gi) * RY) * (long long)BY + j_y) * NZ;
    };

    cf xreg[R0], acc[R0];
    if (a0) {
#pragma unroll
        for (int m = 0; m < R0; ++m) { xreg[m] = load_image(a.x, x_off + jz + PZ::BF0 * m, a.x_planar, b, a.plane); acc[m] = INV ? coil_sum_start(a.aty, x_off + jz + PZ::BF0 * m) : make_float2(0.f, 0.f); }
    }
    issue_s(0);
    // pass 3: the column values of the first coil (one kz column per thread; THREADS >= NZ is not
    // required, further columns are fetched inside the loop)
    cf cnext[RY];
    if (INV && (int)threadIdx.x < NZ) {
        const cf* Vn = v_ptr(0);
#pragma unroll
        for (int k0 = 0; k0 < RY; ++k0) cnext[k0] = Vn[(long long)k0 * BY * NZ + threadIdx.x];
    }

    for (int c = 0; c < a.C; ++c) {
        cf* Vu = v_ptr(c);                                   // + k0 * BY * NZ + kz
        const cf* cS = sS + l * NZ;
        cf v[R0], u[RL];

        if (!INV) {
            cp_async_wait<0>();
            __syncwarp();
            // ---- kz transform of this warp's rows ----
            if (a0) {
#pragma unroll
                for (int m = 0; m < R0; ++m) v[m] = cmul(cS[jz + PZ::BF0 * m], xreg[m]);
            }
            __syncwarp();                                    // S rows consumed: fetch the next coil's
            if (c + 1 < a.C) issue_s(c + 1);
            if (a0) {
                Dft<R0, -1>::run(v);
#pragma unroll
                for (int k = 0; k < R0; ++k) sE[l * WL::EXL + k * PZ::LS1 + jz] = (k == 0) ? v[0] : cmul(v[k], twz[k]);
            }
            __syncwarp();
            if (aL) {
#pragma unroll
                for (int m = 0; m < RL; ++m) u[m] = sE[l * WL::EXL + jz * PZ::LS1 + m];
                Dft<RL, -1>::run(u);
#pragma unroll
                for (int k = 0; k < RL; ++k) sT[m_row * NZ + jz + PZ::BFL * k] = u[k];
            }
            __syncthreads();
            // ---- radix-RY transform across the rows, one kz column per thread ----
            for (int kz = threadIdx.x; kz < NZ; kz += RT::THREADS) {
                cf cvals[RY];
#pragma unroll
                for (int m = 0; m < RY; ++m) cvals[m] = sT[m * NZ + kz];
                Dft<RY, -1>::run(cvals);
#pragma unroll
                for (int k0 = 0; k0 < RY; ++k0) {
                    const cf r = (k0 == 0) ? cvals[0] : cmul(cvals[k0], twy[k0]);
                    Vu[(long long)k0 * BY * NZ + kz] = r;
                }
            }
            __syncthreads();          // the tile is rewritten by the next coil
        } else {
            // ---- inverse radix-RY across the rows ----
            for (int kz = threadIdx.x; kz < NZ; kz += RT::THREADS) {
                cf cvals[RY];
#pragma unroll
                for (int k0 = 0; k0 < RY; ++k0) {
                    const cf r = (kz == (int)threadIdx.x) ? cnext[k0] : Vu[(long long)k0 * BY * NZ + kz];
                    cvals[k0] = (k0 == 0) ? r : cmulc(r, twy[k0]);
                }
                if (kz == (int)threadIdx.x && c + 1 < a.C) {     // next coil's column, in flight during this coil
                    const cf* Vn = v_ptr(c + 1);
#pragma unroll
                    for (int k0 = 0; k0 < RY; ++k0) cnext[k0] = Vn[(long long)k0 * BY * NZ + kz];
                }
                Dft<RY, +1>::run(cvals);
#pragma unroll
                for (int m = 0; m < RY; ++m) sT[m * NZ + kz] = cvals[m];
            }
            __syncthreads();
            // ---- kz inverse of this warp's rows, conjugate-sensitivity coil sum ----
            if (aL) {
#pragma unroll
                for (int k = 0; k < RL; ++k) u[k] = sT[m_row * NZ + jz + PZ::BFL * k];
                Dft<RL, +1>::run(u);
#pragma unroll
                for (int m = 0; m < RL; ++m) sE[l * WL::EXL + jz * PZ::LS1 + m] = u[m];
            }
            cp_async_wait<0>();
            __syncwarp();
            if (a0) {
#pragma unroll
                for (int k = 0; k < R0; ++k) {
                    const cf r = sE[l * WL::EXL + k * PZ::LS1 + jz];
                    v[k] = (k == 0) ? r : cmulc(r, twz[k]);
                }
                Dft<R0, +1>::run(v);
#pragma unroll
                for (int m = 0; m < R0; ++m) {
                    const cf sv = cS[jz + PZ::BF0 * m];
                    acc[m].x = fmaf(sv.x, v[m].x, fmaf(sv.y, v[m].y, acc[m].x));
                    acc[m].y = fmaf(sv.x, v[m].y, fmaf(-sv.y, v[m].x, acc[m].y));
                }
            }
            __syncwarp();                                    // S rows consumed: fetch the next coil's
            if (c + 1 < a.C) issue_s(c + 1);
            __syncthreads();          // tile and exchange area are reused by the next coil
        }
    }
    cp_async_wait<0>();
    if (INV && a0) {
#pragma unroll
        for (int m = 0; m < R0; ++m) {
            const cf av = acc[m];
            store_image(a.out, x_off + jz + PZ::BF0 * m, make_float2(fmaf(-a.eta, av.x, xreg[m].x), fmaf(-a.eta, av.y, xreg[m].y)), a.out_planar, b, a.plane);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// pass 2: radix-BY transform over j, mask and z, inverse; one kz column per thread, no shared memory
// ---------------------------------------------------------------------------------------------
template <int NZ, int RY, int BY, bool HAS_Z>
__global__ void __launch_bounds__(256)
rowtile_mid_kernel(const TileArgs a) {
    constexpr int N1 = RY * BY;
    const int kz = blockIdx.y * blockDim.x + threadIdx.x;          // gridDim.y covers NZ
    const bool col_ok = kz < NZ;
    const unsigned blk = blockIdx.x;                               // (unit, gi, k0)
    const int k0 = (int)(blk % RY);
    const unsigned gi = (blk / RY) % (unsigned)a.G;
    const unsigned unit = blk / (RY * (unsigned)a.G);
    const unsigned bc = unit / (unsigned)a.T;
    const int t = (int)(unit - bc * (unsigned)a.T);
    const int b = (int)(bc / (unsigned)a.C);
    const long long bt = (long long)b * a.T + t;
    const long long pe = (long long)N1 * NZ;
    cf* Vp = a.V + ((((long long)unit * a.G + gi) * RY + k0) * BY) * NZ + kz;   // + j * NZ
    // forward call: the z values of this block's ky group are contiguous in the compact table (ranks
    // zstart[k0] .. zstart[k0+1]); they are staged in shared memory while the transform runs
    // with their scaled squared mask weights; slot ZS_CAP holds zero for the unsampled entries
    constexpr int ZS_CAP = HAS_Z ? 1024 : 1;
    __shared__ cf s_z[ZS_CAP + 1];
    __shared__ float s_w[ZS_CAP + 1];
    int z_first = 0;
    bool z_staged = false;
    if (HAS_Z && a.zstart) {
        z_first = a.zstart[bt * 33 + k0];
        const int nz = a.zstart[bt * 33 + k0 + 1] - z_first;
        z_staged = nz <= ZS_CAP;
        if (z_staged) {
            const cf* zsrc = a.zin + ((long long)unit * a.n0 + a.i0_start + (int)gi) * pe + z_first;
            const float* wsrc = a.m2c + bt * pe + z_first;
            for (int e = threadIdx.x; e < nz; e += blockDim.x) cp_async8(&s_z[e], zsrc + e);
            cp_async_commit();
            for (int e = threadIdx.x; e < nz; e += blockDim.x) s_w[e] = wsrc[e] * a.scale2;
            if (threadIdx.x == 0) { s_z[ZS_CAP] = make_float2(0.f, 0.f); s_w[ZS_CAP] = 0.f; }
        }
    }
    cf c[BY];
    if (col_ok) {
#pragma unroll
        for (int j = 0; j < BY; ++j) c[j] = Vp[(long long)j * NZ];
        Dft<BY, -1>::run(c);
    }
    if (HAS_Z) {
        cp_async_wait<0>();
        __syncthreads();
    }
    if (!col_ok) return;
    const float* mk = a.mask + bt * pe + shift_half(kz, NZ);
    const int i0 = a.i0_start + (int)gi;
    const cf* zz = HAS_Z ? a.zin + ((long long)unit * a.n0 + i0) * pe : nullptr;
    const int* zi = HAS_Z ? a.zidx + bt * pe + kz : nullptr;
    const float* m2 = HAS_Z ? a.m2c + bt * pe : nullptr;
    if (HAS_Z && z_staged) {
        // forward call: weight and z value by rank from shared memory, branch-free (unsampled
        // entries point at the zero slot)
#pragma unroll
        for (int k1 = 0; k1 < BY; ++k1) {
            const int r = zi[(long long)(k0 + RY * k1) * NZ];
            const int e = (r >= 0) ? r - z_first : ZS_CAP;
            const float w = s_w[e];
            const cf q = s_z[e];
            c[k1] = make_float2(fmaf(w, c[k1].x, -q.x), fmaf(w, c[k1].y, -q.y));
        }
    } else {
#pragma unroll
        for (int k1 = 0; k1 < BY; ++k1) {
            const int ky = k0 + RY * k1;                            // raw k index along ky
            if (HAS_Z) {                                            // more sampled entries than the staging area holds
                const int r = zi[(long long)ky * NZ];
                const float w = (r >= 0) ? m2[r] * a.scale2 : 0.f;
                const cf q = (r >= 0) ? zz[r] : make_float2(0.f, 0.f);
                c[k1] = make_float2(fmaf(w, c[k1].x, -q.x), fmaf(w, c[k1].y, -q.y));
            } else {
                const float mv = mk[(long long)shift_half(ky, N1) * NZ];
                c[k1] = cscale(c[k1], mv * mv * a.scale2);
            }
        }
    }
    Dft<BY, +1>::run(c);
#pragma unroll
    for (int j = 0; j < BY; ++j) Vp[(long long)j * NZ] = c[j];
}

// ---------------------------------------------------------------------------------------------
// launch table for the (ky, kz) pairs that have row-tile kernels
// ---------------------------------------------------------------------------------------------
struct PairOps {
    int n1, n2, ry;
    cudaError_t (*fwd)(const TileArgs&, long long images, cudaStream_t);
    cudaError_t (*mid)(const TileArgs&, cudaStream_t);
    cudaError_t (*inv)(const TileArgs&, long long images, cudaStream_t);
};

template <class PZ, int RY, int BY>
struct PairImpl {
    using RT = RowTile<PZ, RY, BY>;
    static_assert(RT::ELIGIBLE, "pair is not eligible for the row-tile kernels");
    template <bool INV> static cudaError_t rows(const TileArgs& a, long long images, cudaStream_t s) {
        static PerDevice done;
        cudaError_t e = ensure_smem(rowtile_kernel<PZ, RY, BY, INV>, RT::SMEM_BYTES, done);
        if (e != cudaSuccess) return e;
        const long long blocks = images * a.G * BY;
        if (blocks <= 0) return cudaSuccess;
        if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
        rowtile_kernel<PZ, RY, BY, INV><<<(unsigned)blocks, RT::THREADS, RT::SMEM_BYTES, s>>>(a);
        return cudaGetLastError();
    }
    static cudaError_t fwd(const TileArgs& a, long long images, cudaStream_t s) { return rows<false>(a, images, s); }
    static cudaError_t inv(const TileArgs& a, long long images, cudaStream_t s) { return rows<true>(a, images, s); }
    static cudaError_t mid(const TileArgs& a, cudaStream_t s) {
        constexpr int NZ = PZ::N;
        const int threads = NZ < 256 ? ((NZ + 31) / 32) * 32 : 256;
        const long long blocks = a.nunits * a.G * RY;
        if (blocks <= 0) return cudaSuccess;
        if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
        dim3 grid((unsigned)blocks, (unsigned)((NZ + threads - 1) / threads));
        if (a.zin) rowtile_mid_kernel<NZ, RY, BY, true><<<grid, threads, 0, s>>>(a);
        else rowtile_mid_kernel<NZ, RY, BY, false><<<grid, threads, 0, s>>>(a);
        return cudaGetLastError();
    }
};

}  // namespace gleam
