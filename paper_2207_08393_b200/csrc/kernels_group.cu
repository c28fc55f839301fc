// Instantiates the kernels of one group of transform lengths (compile with -DGLEAM_GROUP=<g>).
#include "size_ops.cuh"

namespace gleam {
#define GLEAM_SIZE(N, R0, R1, R2, LR, LC) \
    extern const SizeOps size_ops_##N = {N, &SizeImpl<Plan<N, R0, R1, R2>, LR, LC>::row, \
                                         &SizeImpl<Plan<N, R0, R1, R2>, LR, LC>::col};
#include "sizes.def"
#undef GLEAM_SIZE
}  // namespace gleam
