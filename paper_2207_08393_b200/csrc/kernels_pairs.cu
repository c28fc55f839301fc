// Instantiates the row-tile kernels (dc_rowtile.cuh) for one group of the (ky, kz) pairs of pairs.def
// (compile with -DGLEAM_PAIR_GROUP=<g>); group 0 also holds the lookup over all groups.
#include "dc_rowtile.cuh"

#ifndef GLEAM_PAIR_GROUP
#error "compile with -DGLEAM_PAIR_GROUP=<g>"
#endif
#define GLEAM_CAT2(a, b) a##b
#define GLEAM_CAT(a, b) GLEAM_CAT2(a, b)

namespace gleam {

#define GLEAM_PAIR(N1, RY, BY, N2, Z0, Z1) \
    static const PairOps pair_##N1##_##N2 = {N1, N2, RY, &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::fwd, \
                                             &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::mid,          \
                                             &PairImpl<Plan<N2, Z0, Z1, 1>, RY, BY>::inv};
#include "pairs.def"
#undef GLEAM_PAIR

const PairOps* GLEAM_CAT(find_pair_group_, GLEAM_PAIR_GROUP)(int n1, int n2) {
#define GLEAM_PAIR(N1, RY, BY, N2, Z0, Z1) if (n1 == N1 && n2 == N2) return &pair_##N1##_##N2;
#include "pairs.def"
#undef GLEAM_PAIR
    return nullptr;
}

#if GLEAM_PAIR_GROUP == 0
#define GLEAM_PAIR_GROUPS 8
const PairOps* find_pair_group_1(int, int); const PairOps* find_pair_group_2(int, int); const PairOps* find_pair_group_3(int, int);
const PairOps* find_pair_group_4(int, int); const PairOps* find_pair_group_5(int, int); const PairOps* find_pair_group_6(int, int);
const PairOps* find_pair_group_7(int, int);
const PairOps* find_pair(int n1, int n2) {
    const PairOps* (*const groups[GLEAM_PAIR_GROUPS])(int, int) = {find_pair_group_0, find_pair_group_1, find_pair_group_2, find_pair_group_3,
                                                                  find_pair_group_4, find_pair_group_5, find_pair_group_6, find_pair_group_7};
    for (int g = 0; g < GLEAM_PAIR_GROUPS; ++g)
        if (const PairOps* p = groups[g](n1, n2)) return p;
    return nullptr;
}
#endif

}  // namespace gleam
