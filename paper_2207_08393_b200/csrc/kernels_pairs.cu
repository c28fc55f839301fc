// Instantiates the row-tile kernels (dc_rowtile.cuh) for the (ky, kz) pairs listed here.
// GLEAM_PAIR(n1, RY, BY, n2, kz plan R0, R1): ky = n1 = RY * BY, kz = n2 = R0 * R1.
#include "dc_rowtile.cuh"

namespace gleam {

#define GLEAM_PAIRS \
    GLEAM_PAIR(320, 16, 20, 256, 16, 16) \
    GLEAM_PAIR(32, 8, 4, 64, 8, 8)       \
    GLEAM_PAIR(64, 8, 8, 32, 8, 4)       \
    GLEAM_PAIR(320, 16, 20, 64, 8, 8)

#define GLEAM_PAIR(N1, RY, BY, N2, Z0, Z1) \
    static const PairOps pair_##N1##_##N2 = {N1, N2, RY, &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::fwd, \
                                             &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::mid,          \
                                             &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::inv};
GLEAM_PAIRS
#undef GLEAM_PAIR

const PairOps* find_pair(int n1, int n2) {
#define GLEAM_PAIR(N1, RY, BY, N2, Z0, Z1) if (n1 == N1 && n2 == N2) return &pair_##N1##_##N2;
    GLEAM_PAIRS
#undef GLEAM_PAIR
    return nullptr;
}

}  // namespace gleam
