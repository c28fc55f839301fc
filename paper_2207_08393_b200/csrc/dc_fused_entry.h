// Host interface of the fused persistent kernel of the separable 3-D path.
#pragma once
#include <cuda_runtime.h>

namespace gleam {

struct FusedArgs;

// true if the (ky, kz) extents have a fused kernel: kz = 256, ky = 16 * BY for a compiled BY
bool fused3d_supported(int n1, int n2);
cudaError_t fused3d_launch(int n1, const FusedArgs& a, cudaStream_t s);

// test aids: the number of an item that is drawn but never run nor counted (-1: none) and the bound,
// in nanoseconds, of every device-side wait (0 restores the default of two seconds)
int fused3d_withhold();
unsigned long long fused3d_limit_ns();
void fused3d_set_debug(int withhold_item, unsigned long long limit_ns);

}  // namespace gleam
