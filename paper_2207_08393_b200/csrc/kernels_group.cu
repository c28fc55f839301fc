// Instantiates the kernels of one group of transform lengths (compile with -DGLEAM_GROUP=<g>).
#include "size_ops.cuh"

namespace gleam {
#define GLEAM_SIZE(N, A0, A1, A2, LR, B0, B1, B2, LC) \
    extern const SizeOps size_ops_##N = {N, WarpLine<Plan<N, A0, A1, A2>, ROW_FUSED>::ELIGIBLE, &SizeImpl<Plan<N, A0, A1, A2>, LR, Plan<N, B0, B1, B2>, LC>::row, \
                                         &SizeImpl<Plan<N, A0, A1, A2>, LR, Plan<N, B0, B1, B2>, LC>::col};
#include "sizes.def"
#undef GLEAM_SIZE
}  // namespace gleam
