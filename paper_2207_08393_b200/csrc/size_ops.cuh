// Per-length launch table: one entry per supported transform length, defined in the translation
// unit that instantiates the kernels of that length.
#pragma once
#include "dc_kernels.cuh"
#include "dc_warpline.cuh"
#include "dc_warpflat.cuh"
#include "dc_colpipe.cuh"

#include <atomic>

namespace gleam {

// Launch state that CUDA keeps per device (function attributes, occupancy, SM count) is cached per
// device ordinal: one process may drive several GPUs, from several host threads.  The cached values
// are idempotent, so two threads that race on a first use both compute and store the same thing.
constexpr int MAX_DEVICES = 64;
struct PerDevice {
    std::atomic<int> v[MAX_DEVICES];         // 0 = not yet known on that device
    std::atomic<int>* slot() {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
        return &v[dev];
    }
};

struct SizeOps {
    int N;
    bool row_is_warp_resident;   // the ROW kernels of this length derive the sampled ranks themselves
    cudaError_t (*row)(int mode, const RowArgs& a, cudaStream_t s);
    cudaError_t (*col)(int mode, const ColArgs& a, cudaStream_t s);
};

// static_bytes: statically declared shared memory of the kernel, which counts against the same
// 48 KB default limit as the dynamic part
template <class K>
inline cudaError_t ensure_smem(K kernel, size_t bytes, PerDevice& done, size_t static_bytes = 0) {
    if (bytes + static_bytes <= 48 * 1024) return cudaSuccess;
    std::atomic<int>* flag = done.slot();               // null: device ordinal outside the cache, set every time
    if (flag && flag->load(std::memory_order_acquire)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    if (flag) flag->store(1, std::memory_order_release);
    return cudaSuccess;
}

// resident blocks of `kernel` on the current device (SM count x blocks per SM), cached per device
template <class K>
inline cudaError_t resident_slots(K kernel, int threads, size_t smem, PerDevice& cache, int* out) {
    std::atomic<int>* c = cache.slot();
    if (c) { const int v = c->load(std::memory_order_acquire); if (v > 0) { *out = v; return cudaSuccess; } }
    int dev = 0, sms = 0, per_sm = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem)) != cudaSuccess) return e;
    *out = sms * (per_sm > 0 ? per_sm : 1);
    if (c) c->store(*out, std::memory_order_release);
    return cudaSuccess;
}

template <class P, int L, int MODE>
inline cudaError_t launch_row(const RowArgs& a, cudaStream_t s) {
    using E = LineFFT<P, false, L>;
    static PerDevice attr_done;
    cudaError_t e = ensure_smem(row_kernel<P, L, MODE>, E::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    const long long blocks = (a.nrows + L - 1) / L;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
    row_kernel<P, L, MODE><<<(unsigned)blocks, E::THREADS, E::SMEM_BYTES, s>>>(a);
    return cudaGetLastError();
}

// persistent launch of the warp-resident row kernel: one block per resident slot, warps stride
// over the line groups
template <class P, int MODE, bool HAS_Z>
inline cudaError_t launch_warpline_z(const RowArgs& a, cudaStream_t s) {
    using WL = WarpLine<P, MODE, HAS_Z>;
    constexpr int WARPS = 1;
    constexpr size_t SMEM = sizeof(cf) * WARPS * WL::WARP_ELEMS_ALIGNED;
    static PerDevice attr_done;
    static PerDevice slots_cache;
    cudaError_t e = ensure_smem(warpline_kernel<P, WARPS, MODE, HAS_Z>, SMEM, attr_done);
    if (e != cudaSuccess) return e;
    int slots = 0;
    if ((e = resident_slots(warpline_kernel<P, WARPS, MODE, HAS_Z>, WARPS * 32, SMEM, slots_cache, &slots)) != cudaSuccess) return e;
    const long long groups = (a.nrows + WL::LW - 1) / WL::LW;
    long long blocks = (groups + WARPS - 1) / WARPS;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > slots) blocks = slots;
    // one round (every warp takes a single group of lines): the launch may overlap the end of the one before
    return launch_overlapped(groups <= slots, warpline_kernel<P, WARPS, MODE, HAS_Z>, dim3((unsigned)blocks),
                             dim3(WARPS * 32), SMEM, s, a);
}

// GLEAM_NO_SPLIT=1 keeps single-warp blocks for every group (tuning aid, read once).
inline bool split_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("GLEAM_NO_SPLIT"); v = (e && e[0] == '1') ? 0 : 1; }
    return v == 1;
}

// the one-pass kernel with the k-space units numbered across the coils (dc_warpflat.cuh)
template <class P, bool HAS_Z, bool HAS_ATY>
inline cudaError_t launch_warpflat_zy(const RowArgs& a, cudaStream_t s) {
    using WF = WarpFlat<P, HAS_Z, false>;
    static PerDevice attr_done;
    static PerDevice slots_cache;
    cudaError_t e = ensure_smem(warpflat_kernel<P, HAS_Z, false, HAS_ATY>, WF::WARP_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    int slots = 0;
    if ((e = resident_slots(warpflat_kernel<P, HAS_Z, false, HAS_ATY>, 32, WF::WARP_BYTES, slots_cache, &slots)) != cudaSuccess) return e;
    const long long groups = (a.nrows + WF::LW - 1) / WF::LW;
    if (groups <= 0) return cudaSuccess;
    // One round of 8 to 16 groups per SM: one block per SM that holds all its warps.  4 k + 1 (or 4 k + 2) groups per
    // SM: the groups beyond 4 k are split by coils over four warps each, one per scheduler.  (Measured on cine-shaped
    // problems, per call: 13 groups per SM 18.7 -> 16.6 us, 12 per SM 18.7 -> 15.3 us; up to 7 per SM single-warp
    // blocks are faster, 11.3 against 12.7 us.)
    if constexpr (P::RL <= 16 && P::R0 <= 12) {   // larger butterflies need more registers than 16 warps per SM leave
        using WS = WarpFlat<P, HAS_Z, true>;
        static PerDevice attrs_done;
        int sms = 0, dev = 0;
        if (split_enabled() && groups <= slots && cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0 && groups > 7LL * sms) {
            const int per = (int)((groups + sms - 1) / sms);
            int nsplit = (a.C >= 4 && (per % 4 == 1 || per % 4 == 2)) ? per % 4 : 0;
            if (per - nsplit + 4 * nsplit > 16) nsplit = 0;
            const int nwhole = per - nsplit, warps = nwhole + 4 * nsplit;
            const size_t bytes = WS::WARP_BYTES * (size_t)warps;
            // with z the split groups were measured slower than single-warp blocks (13 groups per SM: 25.2 against
            // 24.7 us per call), whole groups alone faster (12 per SM: 22.5 against 24.5 us)
            if (warps <= 16 && bytes <= 227 * 1024 && !(HAS_Z && nsplit > 0)) {
                // the attribute is set once, to what the largest block of this kernel can ask for
                constexpr size_t SMEM_CAP = 227 * 1024;
                if ((e = ensure_smem(warpflat_kernel<P, HAS_Z, true, HAS_ATY>, 16 * WS::WARP_BYTES < SMEM_CAP ? 16 * WS::WARP_BYTES : SMEM_CAP, attrs_done)) != cudaSuccess) return e;
                return launch_overlapped(true, warpflat_kernel<P, HAS_Z, true, HAS_ATY>, dim3((unsigned)sms), dim3(32 * warps), bytes, s, a, nwhole);
            }
        }
    }
    long long blocks = groups;
    if (blocks > slots) blocks = slots;
    return launch_overlapped(groups <= slots, warpflat_kernel<P, HAS_Z, false, HAS_ATY>, dim3((unsigned)blocks), dim3(32), WF::WARP_BYTES, s, a, 1);
}
template <class P, bool HAS_Z>
inline cudaError_t launch_warpflat_z(const RowArgs& a, cudaStream_t s) {
    if constexpr (!HAS_Z) { if (a.aty != nullptr) return launch_warpflat_zy<P, false, true>(a, s); }
    return launch_warpflat_zy<P, HAS_Z, false>(a, s);
}
// GLEAM_NO_FLAT=1 keeps the plain warp-resident kernel for those lengths (tuning aid, read once).
inline bool flat_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("GLEAM_NO_FLAT"); v = (e && e[0] == '1') ? 0 : 1; }
    return v == 1;
}

// Stage plan of the one-pass kernel with units numbered across coils, per length: the last radix RL (8, 16 or
// 32 = butterflies of the first stage per line) where that kernel is used, 0 where the plain plan stays.
// Measured per call against the plain warp-resident kernel (VJP, 4 x 8 coils x 256 rows / 8 x 16 coils x 512 rows):
// 80: 6.8 / 17.4 against 8.6 / 29.3 us; 96: 6.3 / 19.2 against 9.2 / 32.9; 128: 7.4 / 24.7 against 10.2 / 40.3;
// 48: equal for the VJP, forward 24.7 against 33.5; 160 and 320: the cine and brain workloads.
template <int N> struct FlatRL { static constexpr int value = 0; };
template <> struct FlatRL<160> { static constexpr int value = 16; };    // 10 x 16
template <> struct FlatRL<320> { static constexpr int value = 32; };    // 10 x 32
template <> struct FlatRL<128> { static constexpr int value = 16; };    // 8 x 16
template <> struct FlatRL<192> { static constexpr int value = 32; };    // 6 x 32
template <> struct FlatRL<96> { static constexpr int value = 16; };     // 6 x 16
template <> struct FlatRL<80> { static constexpr int value = 16; };     // 5 x 16
template <> struct FlatRL<48> { static constexpr int value = 8; };      // 6 x 8
template <> struct FlatRL<368> { static constexpr int value = 16; };    // 23 x 16
// Which calls of a length take the coil-numbered kernel (1: without z, 2: with z): only where it measured faster.
// 192: the plain plan already keeps most lanes busy (forward 25 against 50 us, but VJP 50 against 46 us on 8 x 16 coils x
// 512 rows); 368 = 23 x 16 (252 registers, 8 warps per SM): VJP 84 against 96 us on knee2d, forward 158 against 153 us.
template <int N> struct FlatCalls { static constexpr int value = (N == 192) ? 2 : (N == 368) ? 1 : 3; };
template <class P> struct FlatPlan {
    static constexpr int RL = FlatRL<P::N>::value;
    using type = Plan<P::N, RL ? P::N / RL : P::R0, RL ? RL : P::R1, RL ? 1 : P::R2>;
};

template <class P, int MODE>
inline cudaError_t launch_warpline(const RowArgs& a, cudaStream_t s) {
    if constexpr (MODE == ROW_FUSED && FlatRL<P::N>::value != 0) {
        using PF = typename FlatPlan<P>::type;
        static_assert(WarpFlat<PF, false>::ELIGIBLE, "not a plan the coil-numbered kernel takes");
        // the numbering across coils pays once a round of 32 units spans more than one coil
        if (flat_enabled() && a.C >= 2 && (FlatCalls<P::N>::value & (a.z != nullptr ? 2 : 1)) != 0)
            return a.z != nullptr ? launch_warpflat_z<PF, true>(a, s) : launch_warpflat_z<PF, false>(a, s);
    }
    if (MODE == ROW_FUSED && a.z != nullptr) return launch_warpline_z<P, MODE, true>(a, s);
    return launch_warpline_z<P, MODE, false>(a, s);
}

template <class P, int L, int MODE>
inline cudaError_t launch_col(const ColArgs& a, cudaStream_t s) {
    using E = LineFFT<P, true, L>;
    static PerDevice attr_done;
    cudaError_t e = ensure_smem(col_kernel<P, L, MODE>, E::SMEM_BYTES, attr_done,
                                MODE == COL_Z ? (COLZ_SELF_MAX + COLZ_SELF_MAX / 32) * sizeof(int) : 0);
    if (e != cudaSuccess) return e;
    long long tiles = (a.es + L - 1) / L;
    ColArgs b = a;
    if (MODE == COL_Z) {
        // the number of sampled ranks is known only on the device: launch a bounded number of blocks
        // per outer index and let them stride over the tiles
        long long cap = 4096 / (a.nouter > 0 ? a.nouter : 1) + 16;
        // blocks that rank the mask row themselves pay for that once each: about eight per SM in all
        if (a.zlist == nullptr) cap = (1184 + a.nouter - 1) / (a.nouter > 0 ? a.nouter : 1);
        if (tiles > cap) tiles = cap;
        b.ztiles = (int)tiles;
    }
    const long long blocks = a.nouter * tiles;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
    col_kernel<P, L, MODE><<<(unsigned)blocks, E::THREADS, E::SMEM_BYTES, s>>>(b);
    return cudaGetLastError();
}

// persistent launch of the pipelined column kernel (separable 3-D path)
template <class P, int L, bool HAS_Z>
inline cudaError_t launch_colpipe_z(const ColArgs& a, cudaStream_t s) {
    using CP = ColPipe<P, L>;
    static PerDevice attr_done;
    static PerDevice slots_cache;
    cudaError_t e = ensure_smem(colpipe_mid_sep_kernel<P, L, HAS_Z>, CP::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    int slots = 0;
    if ((e = resident_slots(colpipe_mid_sep_kernel<P, L, HAS_Z>, CP::THREADS, CP::SMEM_BYTES, slots_cache, &slots)) != cudaSuccess) return e;
    const long long tiles_per_o = (a.es + L - 1) / L;
    const long long tiles = a.nouter * tiles_per_o;
    if (tiles <= 0) return cudaSuccess;
    if (tiles >= 2147483647LL || a.nouter >= 2147483647LL) return cudaErrorInvalidConfiguration;
    // a whole number of rows of tiles_per_o blocks (each block keeps one column tile)
    long long rows = slots / tiles_per_o;
    if (rows < 1) rows = 1;
    if (rows > a.nouter) rows = a.nouter;
    const long long blocks = rows * tiles_per_o;
    colpipe_mid_sep_kernel<P, L, HAS_Z><<<(unsigned)blocks, CP::THREADS, CP::SMEM_BYTES, s>>>(a);
    return cudaGetLastError();
}

template <class P, int L>
inline cudaError_t launch_colpipe(const ColArgs& a, cudaStream_t s) {
    return a.zin ? launch_colpipe_z<P, L, true>(a, s) : launch_colpipe_z<P, L, false>(a, s);
}

template <class P, int LR, class PC, int LC>
struct SizeImpl {
    template <int MODE> static cudaError_t row_mode(const RowArgs& a, cudaStream_t s) {
        if constexpr (WarpLine<P, MODE>::ELIGIBLE) return launch_warpline<P, MODE>(a, s);
        else return launch_row<P, LR, MODE>(a, s);
    }
    static cudaError_t row(int mode, const RowArgs& a, cudaStream_t s) {
        switch (mode) {
            case ROW_FUSED: return row_mode<ROW_FUSED>(a, s);
            case ROW_FWD:   return row_mode<ROW_FWD>(a, s);
            case ROW_INV:   return row_mode<ROW_INV>(a, s);
        }
        return cudaErrorInvalidValue;
    }
    // The plain strided-axis passes of the full-mask path (no k-space work) run faster on wider tiles (16
    // neighbouring lines = 128 contiguous bytes per point row; knee3d col_fwd 808 -> 598 us); the pass with the
    // k-space update measured slower that way (3.4 -> 5.6 ms) and keeps the narrow tile; requesting its mask
    // weights and measurements before the transform cost registers (104 -> 177, one block less per SM) and
    // measured slower on volumes as well.
    static constexpr int LCW = (LC < 16 && sizeof(cf) * (16 * PC::LSZ + 1) <= 100 * 1024 && 16 * PC::MAXBF <= 1024) ? 16 : LC;
    static cudaError_t col(int mode, const ColArgs& a, cudaStream_t s) {
        switch (mode) {
            case COL_Z:        return launch_col<PC, LC, COL_Z>(a, s);
            case COL_MID_SEP:
                if constexpr (ColPipe<PC, LC>::ELIGIBLE) return launch_colpipe<PC, LC>(a, s);
                else return launch_col<PC, LC, COL_MID_SEP>(a, s);
            case COL_MID_FULL: return launch_col<PC, LC, COL_MID_FULL>(a, s);
            case COL_FWD:      return launch_col<PC, LCW, COL_FWD>(a, s);
            case COL_INV:      return launch_col<PC, LCW, COL_INV>(a, s);
            case COL_GRADY:    return launch_col<PC, LC, COL_GRADY>(a, s);
        }
        return cudaErrorInvalidValue;
    }
};

}  // namespace gleam
