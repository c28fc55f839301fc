// Launch helper shared by the kernels that are started with programmatic dependent launch.
#pragma once
#include <cuda_runtime.h>
#include <cstdlib>
#include <utility>

namespace gleam {

// Programmatic dependent launch.  A kernel started through launch_overlapped with allow = true may
// be scheduled while the kernel before it on the stream is still draining; it calls
// grid_dependency_wait() as its first statement, which holds it until that kernel has completed and
// its writes are visible, so only the launch latency and the block start-up overlap.
// grid_launch_dependents() right after the wait lets the next such kernel be scheduled as soon as
// every block of this one has started.  Measured on B200: a gain for launches whose blocks all run
// at once and end together (cine: 8 % per step); a loss of up to 20 % where the launch before has a
// long tail (blocks that take a second group of lines), because the early blocks then sit on the
// SMs next to the tail for tens of microseconds -- so callers allow it for one-round launches only.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// GLEAM_NO_OVERLAP=1 launches these kernels fully serialised (tuning aid, read once).
inline bool overlap_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("GLEAM_NO_OVERLAP"); v = (e && e[0] == '1') ? 0 : 1; }
    return v == 1;
}

template <class... KArgs, class... Args>
inline cudaError_t launch_overlapped(bool allow, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = (allow && overlap_enabled()) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace gleam
