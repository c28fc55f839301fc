// Per-length launch table: one entry per supported transform length, defined in the translation
// unit that instantiates the kernels of that length.
#pragma once
#include "dc_kernels.cuh"

namespace gleam {

struct SizeOps {
    int N;
    cudaError_t (*row)(int mode, const RowArgs& a, cudaStream_t s);
    cudaError_t (*col)(int mode, const ColArgs& a, cudaStream_t s);
};

template <class K>
inline cudaError_t ensure_smem(K kernel, size_t bytes, bool& done) {
    if (!done && bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
    }
    done = true;
    return cudaSuccess;
}

template <class P, int L, int MODE>
inline cudaError_t launch_row(const RowArgs& a, cudaStream_t s) {
    using E = LineFFT<P, false, L>;
    static bool attr_done = false;
    cudaError_t e = ensure_smem(row_kernel<P, L, MODE>, E::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    const long long blocks = (a.nrows + L - 1) / L;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
    row_kernel<P, L, MODE><<<(unsigned)blocks, E::THREADS, E::SMEM_BYTES, s>>>(a);
    return cudaGetLastError();
}

template <class P, int L, int MODE>
inline cudaError_t launch_col(const ColArgs& a, cudaStream_t s) {
    using E = LineFFT<P, true, L>;
    static bool attr_done = false;
    cudaError_t e = ensure_smem(col_kernel<P, L, MODE>, E::SMEM_BYTES, attr_done);
    if (e != cudaSuccess) return e;
    const long long tiles = (a.es + L - 1) / L;
    const long long blocks = a.nouter * tiles;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 2147483647LL) return cudaErrorInvalidConfiguration;
    col_kernel<P, L, MODE><<<(unsigned)blocks, E::THREADS, E::SMEM_BYTES, s>>>(a);
    return cudaGetLastError();
}

template <class P, int LR, class PC, int LC>
struct SizeImpl {
    static cudaError_t row(int mode, const RowArgs& a, cudaStream_t s) {
        switch (mode) {
            case ROW_FUSED: return launch_row<P, LR, ROW_FUSED>(a, s);
            case ROW_FWD:   return launch_row<P, LR, ROW_FWD>(a, s);
            case ROW_INV:   return launch_row<P, LR, ROW_INV>(a, s);
        }
        return cudaErrorInvalidValue;
    }
    static cudaError_t col(int mode, const ColArgs& a, cudaStream_t s) {
        switch (mode) {
            case COL_Z:        return launch_col<PC, LC, COL_Z>(a, s);
            case COL_MID_SEP:  return launch_col<PC, LC, COL_MID_SEP>(a, s);
            case COL_MID_FULL: return launch_col<PC, LC, COL_MID_FULL>(a, s);
            case COL_FWD:      return launch_col<PC, LC, COL_FWD>(a, s);
            case COL_INV:      return launch_col<PC, LC, COL_INV>(a, s);
        }
        return cudaErrorInvalidValue;
    }
};

}  // namespace gleam
