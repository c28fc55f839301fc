// Launch table of the fused persistent kernel of the separable 3-D path (dc_fused3d.cuh).
#include "dc_fused3d.cuh"
#include "dc_fused_entry.h"

#include <atomic>

namespace gleam {

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup: no link-time dependency on the driver
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static std::atomic<EncodeTiledFn> cached{nullptr};
    EncodeTiledFn fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
            cudaGetLastError();
            return nullptr;
        }
        fn = (EncodeTiledFn)p;
        cached.store(fn, std::memory_order_release);
    }
    return fn;
}

// 4-D map (d0 fastest) over a dense array of `elem`-byte values, box (b0, 1, b2, 1)
static cudaError_t make_map(CUtensorMap* tm, const void* base, CUtensorMapDataType type, size_t elem, uint64_t d0, uint64_t d1,
                            uint64_t d2, uint64_t d3, uint64_t s1, uint64_t s2, uint64_t s3, uint32_t b0, uint32_t b2) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return cudaErrorNotSupported;
    const cuuint64_t dims[4] = {d0, d1, d2, d3};
    const cuuint64_t strides[3] = {s1 * elem, s2 * elem, s3 * elem};        // bytes; dimension 0 is dense
    const cuuint32_t box[4] = {b0, 1, b2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = fn(tm, type, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int BY>
static cudaError_t launch_fused(const FusedArgs& a, cudaStream_t s) {
    constexpr uint64_t NZ = fused::NZ, RY = fused::RY, N1 = RY * BY;
    const uint64_t images = (uint64_t)a.nslabs / a.n0;                       // B T
    const uint64_t sens_slabs = images / a.T * a.C * a.Ts * a.n0;            // B C Ts n0
    CUtensorMap tm_sens, tm_x, tm_ring, tm_mask;
    cudaError_t me;
    if ((me = make_map(&tm_sens, a.sens, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 8, NZ, BY, RY, sens_slabs, NZ, BY * NZ, N1 * NZ, NZ, RY)) != cudaSuccess) return me;
    if ((me = make_map(&tm_x, a.x, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 8, NZ, BY, RY, (uint64_t)a.nslabs, NZ, BY * NZ, N1 * NZ, NZ, RY)) != cudaSuccess) return me;
    if ((me = make_map(&tm_ring, a.W, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 8, NZ, BY, RY, (uint64_t)a.R * a.C, NZ, BY * NZ, N1 * NZ, NZ, RY)) != cudaSuccess) return me;
    if ((me = make_map(&tm_mask, a.mask, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, NZ, RY, BY, images, NZ, RY * NZ, N1 * NZ, NZ, BY)) != cudaSuccess) return me;
    static PerDevice attr_done, sm_cache;
    cudaError_t e;
    if (a.zin) {
        if ((e = ensure_smem(fused3d_kernel<BY, true>, fused::SMEM_BYTES, attr_done)) != cudaSuccess) return e;
    }
    static PerDevice attr_done_v;
    if ((e = ensure_smem(fused3d_kernel<BY, false>, fused::SMEM_BYTES, attr_done_v)) != cudaSuccess) return e;
    int blocks = 0;
    if ((e = resident_slots(fused3d_kernel<BY, false>, fused::THREADS, fused::SMEM_BYTES, sm_cache, &blocks)) != cudaSuccess) return e;
    const long long items = (long long)(a.nslabs + a.L3) * (2 * BY + fused::RY);
    if (blocks > items) blocks = (int)items;
    if (blocks < 1) return cudaSuccess;
    if (a.zin) fused3d_kernel<BY, true><<<blocks, fused::THREADS, fused::SMEM_BYTES, s>>>(a, tm_sens, tm_x, tm_ring, tm_mask);
    else fused3d_kernel<BY, false><<<blocks, fused::THREADS, fused::SMEM_BYTES, s>>>(a, tm_sens, tm_x, tm_ring, tm_mask);
    return cudaGetLastError();
}

#define GLEAM_FUSED_BYS GLEAM_FUSED_BY(4) GLEAM_FUSED_BY(8) GLEAM_FUSED_BY(20)

bool fused3d_supported(int n1, int n2) {
    if (n2 != fused::NZ || n1 % fused::RY != 0) return false;
    switch (n1 / fused::RY) {
#define GLEAM_FUSED_BY(B) case B: return true;
        GLEAM_FUSED_BYS
#undef GLEAM_FUSED_BY
        default: return false;
    }
}

cudaError_t fused3d_launch(int n1, const FusedArgs& a, cudaStream_t s) {
    switch (n1 / fused::RY) {
#define GLEAM_FUSED_BY(B) case B: return launch_fused<B>(a, s);
        GLEAM_FUSED_BYS
#undef GLEAM_FUSED_BY
        default: return cudaErrorInvalidValue;
    }
}

// test aids (process-wide): an item whose completion is withheld, and a shorter bound of the waits
static std::atomic<int> g_withhold{-1};
static std::atomic<unsigned long long> g_limit_ns{2000000000ull};
int fused3d_withhold() { return g_withhold.load(); }
unsigned long long fused3d_limit_ns() { return g_limit_ns.load(); }
void fused3d_set_debug(int withhold_item, unsigned long long limit_ns) {
    g_withhold.store(withhold_item);
    g_limit_ns.store(limit_ns ? limit_ns : 2000000000ull);
}

}  // namespace gleam
