// One persistent kernel for the separable 3-D path: the three passes of dc_rowtile.cuh run as a
// dataflow over readout slabs, so that the coil workspace of a slab lives in L2 between its passes
// instead of streaming through HBM three times.
//
// ky = N1 = RY * BY (RY = 16), kz = NZ = 256 = 16 * 16.  Image-side ky = j + BY m (m < RY), k-space
// ky = k0 + RY k1 (k1 < BY).  Work items, per readout slab s (an image b,t and a readout index):
//   P1(s, j)   rows ky = j + BY m of every coil: S_c x, radix-RY transform across the rows, kz
//              transform of each result row, store  W[slot][c][k0][j][kz]
//   P2(s, k0)  the BY contiguous rows of (c, k0): twiddle w_N1^(j k0), radix-BY transform over j,
//              mask^2 / (N1 NZ) (and - z in the forward call), inverse, conjugate twiddle, in place
//   P3(s, j)   mirror of P1: kz inverse, inverse radix-RY, conj(S_c) coil sum, out = x - eta sum
// P2(s,.) needs all P1(s,.), P3(s,.) needs all P2(s,.); W is a ring of R slabs, so P1(s,.) also
// needs all P3(s-R,.).  Items are drawn from one global counter in the order
//   period p:  P3(p - L3, j) for all j | P2(p - L2, k0) for all k0 | P1(p, j) for all j
// so every dependency of an item has a smaller number: whoever drew it is already running, and
// nothing requires the blocks to be co-resident.  Completion is counted per slab in global memory
// (release / acquire); every wait on such a counter and on a shared-memory barrier is bounded: after
// the limit the block raises the error word, stops starting work, and the host reports
// GLEAM_ERR_TIMEOUT from gleam_dc_check_status.
//
// Block = two compute groups of 256 threads that take half of the coils of an item each (the coil sum
// of P3 is completed through shared memory in a fixed order) and a producer warpgroup with one elected
// lane per group: the first draws the items; each polls the item's dependency and stages the input
// tiles of its group one step ahead with tiled TMA copies (cp.async.bulk.tensor + mbarrier) while the
// group computes.  A group owns three 32 KB buffers A | B | C.  The transposition between the row-wise
// and the column-wise transform happens in place in the staged tile itself (a thread rewrites the column
// it read; a warp rewrites its own two rows with an XOR-swizzled 16 x 16 exchange), so a step needs one
// group-wide barrier, and the tile of step s + 1 arrives in the other buffer meanwhile:
//   P1  x tile -> C once; S tiles alternate A, B      P2  BY rows -> A | B (+ mask rows once)
//   P3  W tiles alternate B, C; S tile -> A; the x rows for the update follow in the W alternation
#pragma once
#include "size_ops.cuh"
#include <cuda.h>          // CUtensorMap (type only; the encoder is looked up at run time)

namespace gleam {

struct FusedArgs {
    const cf* x; const cf* sens; cf* out;     // image side
    cf* W;                                    // ring (R, C, RY, BY, NZ)
    const float* mask;                        // (B,T,N1,NZ)
    const cf* zin; const int* zidx;           // forward call: compact z table, rank map
    const float* m2c; const int* zstart;      //               squared weights by rank, first rank of each ky-mod-RY group
    int* ctrl;                                // [0] next item, [1] error word; per-slab counters from ctrl + 64
    float eta, scale2;
    int C, T, Ts, n0;
    int nslabs;                               // B*T*n0
    int R, L2, L3;                            // ring slots and the lags of P2 / P3 behind P1 (slabs)
    int withhold;                             // test aid: this item is drawn but neither run nor counted (-1: none)
    unsigned long long limit_ns;              // bound of every wait
};

namespace fused {

constexpr int NZ = 256, RY = 16, GT = 256;
constexpr int CONSUMERS = 2 * GT, THREADS = CONSUMERS + 128;   // four compute warpgroups + the producer's
constexpr int REGS_PRODUCER = 24, REGS_COMPUTE = 112;           // register split after the kernel has started
constexpr int TILE = RY * NZ;                             // complex values of a staged tile (32 KB)
constexpr int GROUP_ELEMS = 3 * TILE;                     // A | B | C
constexpr size_t SMEM_BYTES = sizeof(cf) * 2 * GROUP_ELEMS + 256;

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long gtimer() {
    unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v; asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
    int v; asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void red_release(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// global -> shared bulk copy that reports its bytes to an mbarrier; addresses and size are multiples of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// One tiled TMA copy of a 4-D box (coordinates innermost first; c0 is always 0 here, so the 16-byte rule
// on the innermost coordinate holds).  The tensor maps cover this GPU's own memory only.
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3,
                                            unsigned long long* bar) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(void* dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3,
                                                 unsigned long long* bar, unsigned long long policy) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ void named_bar(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void st_keep(cf* p, cf v, unsigned long long pol) {      // workspace store, kept in L2
    asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1,%2}, %3;" ::"l"(p), "f"(v.x), "f"(v.y), "l"(pol) : "memory");
}

// Bounded wait on a shared-memory barrier.  `stop` is a shared flag raised by whoever gave up first.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, const volatile int* stop,
                                          unsigned long long limit_ns, const volatile int* stop2 = nullptr) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = gtimer();
    for (;;) {
        if (mbar_try(bar, parity)) return true;
        if (*stop != 0 || (stop2 != nullptr && *stop2 != 0)) return false;
        if (gtimer() - t0 > limit_ns) return false;
    }
}

struct Shared {                      // control block behind the tiles
    unsigned long long full[2][3], empty[2][3];       // [group][A / B / C]
    unsigned long long item_full[2], item_empty[2];
    int item[2];                                      // item number of the slot (bit 30: withheld)
    int dead[2];                                      // group gave up (sticky)
    int prod_dead;                                    // producer gave up (sticky)
    int stop_flag[2];                                 // written during item k (slot k & 1), read after its closing barrier
};

}  // namespace fused

template <int BY, bool HAS_Z>
__global__ void __launch_bounds__(fused::THREADS, 1)
fused3d_kernel(const FusedArgs a, const __grid_constant__ CUtensorMap tm_sens, const __grid_constant__ CUtensorMap tm_x,
               const __grid_constant__ CUtensorMap tm_ring, const __grid_constant__ CUtensorMap tm_mask) {
    // tensor maps (64-bit elements for the complex arrays), all with box (NZ, 1, RY, 1) except the mask:
    //   tm_sens (NZ, BY, RY, B C Ts n0)   rows ky = j + BY m of one slab of one coil: coordinates (0, j, 0, unit n0 + i0)
    //   tm_x    (NZ, BY, RY, B T n0)      the same rows of x: (0, j, 0, slab)
    //   tm_ring (NZ, BY, RY, R C)         rows (k0, j) for all k0 of one coil of a ring slot: (0, j, 0, slot C + c)
    //   tm_mask (NZ, RY, BY, B T) float   rows k0 + RY k1 for all k1, box (NZ, 1, BY, 1): (0, k0, 0, image)
    using namespace fused;
    constexpr int N1 = RY * BY;
    static_assert(BY >= 2 && BY <= 24 && BY % 2 == 0, "radix of the middle pass (even: the half shift of ky keeps ky mod RY)");
    // The mask rows of the middle pass arrive on buffer B's barrier and are guarded by B's release, so they have to
    // lie in B's part of the shared memory: behind the tile rows that spill into B (BY > RY), else at B's start.  (At
    // gbase + BY * NZ they lay inside buffer A for BY < RY, where a block that went from a third-pass item straight to a
    // middle-pass item had them written over the partial coil sums still kept in A.)
    constexpr int MASK_OFF = BY * NZ > TILE ? BY * NZ : TILE;
    static_assert(MASK_OFF >= TILE && MASK_OFF * 8 + BY * NZ * 4 <= 2 * TILE * 8, "mask rows of the middle pass fit buffer B");
    extern __shared__ __align__(128) float2 fsmem[];
    float2* const smem = fsmem;
    Shared* sh = reinterpret_cast<Shared*>(smem + 2 * GROUP_ELEMS);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int g = 0; g < 2; ++g)
            for (int b = 0; b < 3; ++b) { mbar_init(&sh->full[g][b], 1); mbar_init(&sh->empty[g][b], GT / 32); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sh->item_full[s], 1); mbar_init(&sh->item_empty[s], 3); sh->stop_flag[s] = 0; }
        sh->dead[0] = sh->dead[1] = 0; sh->prod_dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int per_period = BY + RY + BY;
    const long long total = (long long)(a.nslabs + a.L3) * per_period;
    const int n_g[2] = {(a.C + 1) / 2, a.C / 2};              // coils of group 0 / 1
    const long long slab_elems = (long long)N1 * NZ;
    int* c1 = a.ctrl + 64; int* c2 = c1 + a.nslabs; int* c3 = c2 + a.nslabs;
    unsigned long long* stats = reinterpret_cast<unsigned long long*>(a.ctrl + 8);

    // The launch gives every thread floor(65536 / 640 / 8) * 8 = 96 registers; the producers' warpgroup
    // hands most of its share back and the compute warpgroups take 112 each:
    // 128 * 24 + 512 * 112 = 60416 <= 640 * 96 = 61440.
    static_assert(128 * REGS_PRODUCER + CONSUMERS * REGS_COMPUTE <= THREADS * 96, "register split exceeds the launch's registers");
    if (warp >= CONSUMERS / 32) {
        // =================================== producers ===================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_PRODUCER));
        const int g = warp - CONSUMERS / 32;                   // the producer of group g is lane 0 of producer warp g
        if (g > 1 || lane != 0) return;
        unsigned nfill[3] = {0, 0, 0};
        cf* const gbase = smem + g * GROUP_ELEMS;
        unsigned long long pol_first, pol_last;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_last));
        const int n = n_g[g], c_first = g * n_g[0];

        // arms the barrier of the next fill of buffer b once the group has released the fill before
        auto begin_fill = [&](int b, unsigned bytes) -> bool {
            const unsigned f = nfill[b];
            if (f > 0 && !mbar_wait(&sh->empty[g][b], (f - 1) & 1, &sh->dead[g], a.limit_ns, &sh->prod_dead)) return false;
            mbar_expect_tx(&sh->full[g][b], bytes);
            nfill[b] = f + 1;
            return true;
        };
        // time spent waiting and number of waits that had to spin, per kind (ctrl + 8: pairs of 64-bit words):
        // 0 ring slot free (P1), 1 first pass of the slab complete (P2), 2 middle pass complete (P3)
        auto wait_counter = [&](const int* ctr, int target, int kind) -> bool {
            if (ld_acquire(ctr) >= target) return true;
            const unsigned long long t0 = gtimer();
            bool ok = false;
            for (;;) {
                if (ld_acquire(ctr) >= target) { ok = true; break; }
                if (ld_relaxed(a.ctrl + 1) != 0 || *(volatile int*)&sh->prod_dead != 0) break;
                if (gtimer() - t0 > a.limit_ns) break;
                __nanosleep(64);
            }
            atomicAdd(stats + 2 * kind, gtimer() - t0);
            atomicAdd(stats + 2 * kind + 1, 1ull);
            return ok;
        };
        auto sens_slab = [&](int gs, int c) -> int {           // last coordinate of tm_sens: S_c of slab gs
            const int bt = gs / a.n0, i0 = gs - bt * a.n0;
            const int b = bt / a.T, t = bt - b * a.T;
            return ((b * a.C + c) * a.Ts + (a.Ts > 1 ? t : 0)) * a.n0 + i0;
        };

        bool ok = true;
        for (unsigned k = 0; ok; ++k) {
            const int slot = k & 1;
            int word;
            if (g == 0) {
                // draw the next item and publish it to both groups and to the other producer
                long long id = atomicAdd(a.ctrl, 1);
                if (id > total) id = total;
                word = (int)id;
                if (id < total && a.withhold >= 0 && id == a.withhold) word |= 1 << 30;
                if (k >= 2 && !mbar_wait(&sh->item_empty[slot], ((k >> 1) - 1) & 1, &sh->dead[0], a.limit_ns, &sh->dead[1])) { ok = false; break; }
                sh->item[slot] = word;
                mbar_arrive(&sh->item_full[slot]);
            } else {
                if (!mbar_wait(&sh->item_full[slot], (k >> 1) & 1, &sh->prod_dead, a.limit_ns, &sh->dead[1])) { ok = false; break; }
                word = *(volatile int*)&sh->item[slot];
                mbar_arrive(&sh->item_empty[slot]);
            }
            const long long id = word & ~(1 << 30);
            if (id >= total) break;
            if (word >> 30) continue;
            const int period = (int)(id / per_period), q = (int)(id % per_period);
            if (q < BY) {
                // ---- P3(gs, j): per step W tile -> B / C alternating, S tile -> A; then the x tile in the W alternation
                const int gs = period - a.L3, j = q;
                if (gs < 0 || gs >= a.nslabs) continue;
                ok = wait_counter(c2 + gs, RY, 2);
                asm volatile("fence.proxy.async;" ::: "memory");
                const int rs = gs % a.R;
                for (int s = 0; ok && s < n; ++s) {
                    const int wb = 1 + (s & 1);
                    if (!(ok = begin_fill(wb, TILE * 8))) break;
                    tma_load_4d_hint(gbase + wb * TILE, &tm_ring, 0, j, 0, rs * a.C + c_first + s, &sh->full[g][wb], pol_first);
                    if (!(ok = begin_fill(0, TILE * 8))) break;
                    tma_load_4d_hint(gbase, &tm_sens, 0, j, 0, sens_slab(gs, c_first + s), &sh->full[g][0], pol_first);
                }
                if (ok) {
                    const int xb = 1 + (n & 1);
                    if ((ok = begin_fill(xb, TILE * 8))) tma_load_4d_hint(gbase + xb * TILE, &tm_x, 0, j, 0, gs, &sh->full[g][xb], pol_first);
                }
            } else if (q < BY + RY) {
                // ---- P2(gs, k0): per step the BY rows of (c, k0) -> A | B; with the first step the mask rows behind them
                const int gs = period - a.L2, k0 = q - BY;
                if (gs < 0 || gs >= a.nslabs) continue;
                ok = wait_counter(c1 + gs, BY, 1);
                asm volatile("fence.proxy.async;" ::: "memory");
                const int rs = gs % a.R;
                const int bt = gs / a.n0;
                constexpr int ROWS_A = BY < RY ? BY : RY, ROWS_B = BY - ROWS_A;
                for (int s = 0; ok && s < n; ++s) {
                    const cf* src = a.W + (((long long)rs * a.C + c_first + s) * RY + k0) * BY * NZ;
                    const unsigned bytes_b = ROWS_B * NZ * 8 + (s == 0 ? BY * NZ * 4 : 0);
                    if (bytes_b > 0) {
                        if (!(ok = begin_fill(1, bytes_b))) break;
                        if (ROWS_B > 0) bulk_load(gbase + TILE, src + ROWS_A * NZ, ROWS_B * NZ * 8, &sh->full[g][1]);
                        if (s == 0) tma_load_4d(gbase + MASK_OFF, &tm_mask, 0, k0, 0, bt, &sh->full[g][1]);
                    }
                    if (!(ok = begin_fill(0, ROWS_A * NZ * 8))) break;
                    bulk_load(gbase, src, ROWS_A * NZ * 8, &sh->full[g][0]);
                }
            } else {
                // ---- P1(gs, j): x tile -> C, then per step S tile -> A / B alternating
                const int gs = period, j = q - BY - RY;
                if (gs >= a.nslabs || n == 0) continue;
                if (gs >= a.R) ok = wait_counter(c3 + gs - a.R, BY, 0);
                if (ok && (ok = begin_fill(2, TILE * 8))) tma_load_4d(gbase + 2 * TILE, &tm_x, 0, j, 0, gs, &sh->full[g][2]);
                for (int s = 0; ok && s < n; ++s) {
                    const int sb = s & 1;
                    if (!(ok = begin_fill(sb, TILE * 8))) break;
                    tma_load_4d(gbase + sb * TILE, &tm_sens, 0, j, 0, sens_slab(gs, c_first + s), &sh->full[g][sb]);
                }
            }
        }
        if (!ok) {                                   // gave up: raise the error word, tell everyone in the block
            atomicExch(a.ctrl + 1, 1);
            sh->prod_dead = 1;
        }
        // copies that were started must have landed before the block may end
        for (int b = 0; b < 3; ++b)
            if (nfill[b] > 0) {
                volatile int never = 0;
                mbar_wait(&sh->full[g][b], (nfill[b] - 1) & 1, &never, a.limit_ns);
            }
        return;
    }

    // =================================== compute groups ===================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_COMPUTE));
    const int g = warp >> 3;                       // group
    const int gt = tid & (GT - 1);                 // thread of the group
    const int r = gt >> 4, a16 = gt & 15;          // row-owned layout: row, and position in the 16 x 16 split of kz
    cf* const gbase = smem + g * GROUP_ELEMS;      // A | B | C
    cf* const obase = smem + (g ^ 1) * GROUP_ELEMS;
    const int gbar = 1 + g;
    unsigned nuse[3] = {0, 0, 0};                  // fills of A / B / C consumed so far
    bool dead = false;                             // the whole group shares this value at every barrier
    unsigned long long keep_policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep_policy));

    // every warp waits for the next fill of buffer b through its first lane (bounded); a warp that gave up keeps
    // running the same control flow without waiting and without storing
    auto wait_full = [&](int b) {
        int failed = 0;
        if (lane == 0 && !dead) {
            if (!mbar_try(&sh->full[g][b], nuse[b] & 1)) {
                const unsigned long long t0 = gtimer();
                if (!mbar_wait(&sh->full[g][b], nuse[b] & 1, &sh->prod_dead, a.limit_ns, &sh->dead[g])) { sh->dead[g] = 1; failed = 1; }
                if (gt == 0) {                                   // not landed when needed: count the wait (kinds 3: A, 4: B or C)
                    atomicAdd(stats + 2 * (b == 0 ? 3 : 4), gtimer() - t0);
                    atomicAdd(stats + 2 * (b == 0 ? 3 : 4) + 1, 1ull);
                }
            }
        }
        dead = dead || (__shfl_sync(0xffffffffu, failed, 0) != 0);
        ++nuse[b];
    };
    auto release = [&](int b) {                    // this warp has finished with the buffer
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->empty[g][b]);
    };
    auto group_sync = [&]() {
        named_bar(gbar, GT);
        dead = dead || (*(volatile int*)&sh->dead[g] != 0);
    };
    // 16 x 16 exchange inside one row of 256 values, conflict-free without padding: element (p, q) lives at 16 p + (q ^ p)
    auto xs = [&](int p, int q) -> int { return 16 * p + (q ^ p); };

    for (unsigned k = 0;; ++k) {
        const int slot = k & 1;
        if (gt == 0) {
            if (!dead && !mbar_wait(&sh->item_full[slot], (k >> 1) & 1, &sh->prod_dead, a.limit_ns)) sh->dead[g] = 1;
        }
        group_sync();
        const int word = dead ? (int)total : *(volatile int*)&sh->item[slot];
        __syncwarp();
        if (gt == 0 && !dead) mbar_arrive(&sh->item_empty[slot]);
        const long long id = word & ~(1 << 30);
        const bool withheld = (word >> 30) & 1;
        if (id >= total) {
            // two closing barriers like every item, so that both groups leave together
            if (dead && gt == 0) sh->stop_flag[slot] = 1;
            named_bar(3, CONSUMERS);
            named_bar(3, CONSUMERS);
            break;
        }
        const int period = (int)(id / per_period), q = (int)(id % per_period);
        int* done_ctr = nullptr;
        bool release_a_after_close = false;
        const int n = n_g[g], c_first = g * n_g[0];

        if (q < BY) {
            // ------------------------------ P3(gs, j) ------------------------------
            const int gs = period - a.L3;
            const bool live = !withheld && gs >= 0 && gs < a.nslabs;
            if (live) {
                cf acc[RY];
#pragma unroll
                for (int m = 0; m < RY; ++m) acc[m] = make_float2(0.f, 0.f);
                cf twz[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) twz[e] = unit_root_fwd<NZ>((a16 * e) % NZ);
                cf* const S = gbase;
                for (int s = 0; s < n; ++s) {
                    const int wb = 1 + (s & 1);
                    cf* const row = gbase + wb * TILE + r * NZ;          // this thread's row of the W tile
                    wait_full(wb);         // the column reads of the step before used the other W buffer
                    // ---- kz inverse of the warp's two rows, in place ----
                    cf w[16];
#pragma unroll
                    for (int k1 = 0; k1 < 16; ++k1) w[k1] = row[a16 + 16 * k1];
                    Dft<16, +1>::run(w);                               // k1 -> a'
#pragma unroll
                    for (int e = 1; e < 16; ++e) w[e] = cmulc(w[e], twz[e]);
                    __syncwarp();
#pragma unroll
                    for (int e = 0; e < 16; ++e) row[xs(a16, e)] = w[e];
                    __syncwarp();
                    cf u[16];
#pragma unroll
                    for (int k2 = 0; k2 < 16; ++k2) u[k2] = row[xs(k2, a16)];
                    Dft<16, +1>::run(u);                               // k2 -> b
                    __syncwarp();
#pragma unroll
                    for (int b = 0; b < 16; ++b) row[a16 + 16 * b] = u[b];
                    wait_full(0);
                    named_bar(gbar, GT);
                    // ---- inverse radix-RY across the rows, conj(S) and the coil sum: one kz position per thread ----
                    cf v[RY];
                    const cf* const col = gbase + wb * TILE + gt;
#pragma unroll
                    for (int k0 = 0; k0 < RY; ++k0) v[k0] = col[k0 * NZ];
                    release(wb);
                    Dft<RY, +1>::run(v);                               // k0 -> m
#pragma unroll
                    for (int m = 0; m < RY; ++m) {
                        const cf sv = S[m * NZ + gt];
                        acc[m].x = fmaf(sv.x, v[m].x, fmaf(sv.y, v[m].y, acc[m].x));
                        acc[m].y = fmaf(sv.x, v[m].y, fmaf(-sv.y, v[m].x, acc[m].y));
                    }
                    if (s + 1 < n) release(0);          // after the last step buffer A carries the partial sums below
                }
                // partial coil sums of this group into buffer A (a thread only touches its own column), x tile in the W alternation
                if (n > 0) {
#pragma unroll
                    for (int m = 0; m < RY; ++m) S[m * NZ + gt] = acc[m];
                } else {
#pragma unroll
                    for (int m = 0; m < RY; ++m) S[m * NZ + gt] = make_float2(0.f, 0.f);
                }
                wait_full(1 + (n & 1));
            }
            if (dead && gt == 0) sh->stop_flag[slot] = 1;
            named_bar(3, CONSUMERS);
            dead = dead || (*(volatile int*)&sh->dead[g] != 0);
            if (live) {
                // group g completes rows m in [g RY/2, (g+1) RY/2): group 0's partial sum + group 1's, then the update
                const cf* P0 = g == 0 ? gbase : obase;
                const cf* P1 = g == 0 ? obase : gbase;
                const cf* X = gbase + (1 + (n & 1)) * TILE;
                const long long xo = (long long)gs * slab_elems + (long long)q * NZ + gt;
#pragma unroll
                for (int mm = 0; mm < RY / 2; ++mm) {
                    const int m = g * (RY / 2) + mm;
                    const cf p0 = P0[m * NZ + gt], p1 = P1[m * NZ + gt];
                    const cf xv = X[m * NZ + gt];
                    const float sx = p0.x + p1.x, sy = p0.y + p1.y;
                    if (!dead) a.out[xo + (long long)BY * m * NZ] = make_float2(fmaf(-a.eta, sx, xv.x), fmaf(-a.eta, sy, xv.y));
                }
                release(1 + (n & 1));
                done_ctr = c3 + gs;
                release_a_after_close = n > 0;      // the other group reads this group's partial sums until the closing barrier
            }
        } else if (q < BY + RY) {
            // ------------------------------ P2(gs, k0) ------------------------------
            const int gs = period - a.L2, k0 = q - BY;
            const bool live = !withheld && gs >= 0 && gs < a.nslabs;
            if (live && n > 0) {
                const int rs = gs % a.R;
                cf twy[BY];
#pragma unroll
                for (int j = 0; j < BY; ++j) twy[j] = unit_root_fwd<N1>((j * k0) % N1);
                float wts[BY];
                const float* mrows = reinterpret_cast<const float*>(gbase + MASK_OFF);
                for (int s = 0; s < n; ++s) {
                    const int c = c_first + s;
                    wait_full(0);
                    if (BY > RY || s == 0) wait_full(1);
                    cf cv[BY];
#pragma unroll
                    for (int j = 0; j < BY; ++j) cv[j] = gbase[j * NZ + gt];        // rows beyond RY continue into buffer B
                    if (s == 0) {
#pragma unroll
                        for (int k1 = 0; k1 < BY; ++k1) {         // the staged rows are ky = k0 + RY k1' in natural order; the raw index needs the half shift
                            const float mv = mrows[((k1 + BY / 2) % BY) * NZ + shift_half(gt, NZ)];
                            wts[k1] = mv * mv * a.scale2;
                        }
                    }
                    release(0);
                    if (BY > RY || s == 0) release(1);
#pragma unroll
                    for (int j = 1; j < BY; ++j) cv[j] = cmul(cv[j], twy[j]);
                    Dft<BY, -1>::run(cv);                               // j -> k1
#pragma unroll
                    for (int k1 = 0; k1 < BY; ++k1) cv[k1] = cscale(cv[k1], wts[k1]);
                    Dft<BY, +1>::run(cv);                               // k1 -> j
#pragma unroll
                    for (int j = 1; j < BY; ++j) cv[j] = cmulc(cv[j], twy[j]);
                    cf* dst = a.W + (((long long)rs * a.C + c) * RY + k0) * BY * NZ + gt;
                    if (!dead) {
#pragma unroll
                        for (int j = 0; j < BY; ++j) st_keep(dst + j * NZ, cv[j], keep_policy);
                    }
                }
            }
            if (live) done_ctr = c2 + gs;
            if (dead && gt == 0) sh->stop_flag[slot] = 1;
            named_bar(3, CONSUMERS);
        } else {
            // ------------------------------ P1(gs, j) ------------------------------
            const int gs = period, j = q - BY - RY;
            const bool live = !withheld && gs < a.nslabs;
            if (live && n > 0) {
                const int rs = gs % a.R;
                cf twz[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) twz[e] = unit_root_fwd<NZ>((a16 * e) % NZ);
                wait_full(2);
                cf xr[RY];
#pragma unroll
                for (int m = 0; m < RY; ++m) xr[m] = gbase[2 * TILE + m * NZ + gt];
                release(2);
                for (int s = 0; s < n; ++s) {
                    const int c = c_first + s, sb = s & 1;
                    cf* const tile = gbase + sb * TILE;
                    wait_full(sb);
                    // ---- S x and the radix-RY transform across the rows: one kz position per thread, in place ----
                    cf v[RY];
#pragma unroll
                    for (int m = 0; m < RY; ++m) v[m] = cmul(tile[m * NZ + gt], xr[m]);
                    Dft<RY, -1>::run(v);                               // m -> k0
#pragma unroll
                    for (int k0 = 0; k0 < RY; ++k0) tile[k0 * NZ + gt] = v[k0];
                    named_bar(gbar, GT);
                    // ---- kz transform of the warp's two rows, in place, then out to the ring ----
                    cf* const row = tile + r * NZ;
                    cf u[16];
#pragma unroll
                    for (int b = 0; b < 16; ++b) u[b] = row[a16 + 16 * b];
                    Dft<16, -1>::run(u);                               // b -> k2
#pragma unroll
                    for (int e = 1; e < 16; ++e) u[e] = cmul(u[e], twz[e]);
                    __syncwarp();
#pragma unroll
                    for (int k2 = 0; k2 < 16; ++k2) row[xs(k2, a16)] = u[k2];
                    __syncwarp();
                    cf w[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) w[e] = row[xs(a16, e)];
                    release(sb);
                    Dft<16, -1>::run(w);                               // a' -> k1
                    cf* dst = a.W + ((((long long)rs * a.C + c) * RY + r) * BY + j) * NZ + a16;
                    if (!dead) {
#pragma unroll
                        for (int k1 = 0; k1 < 16; ++k1) st_keep(dst + 16 * k1, w[k1], keep_policy);
                    }
                }
            }
            if (live) done_ctr = c1 + gs;
            if (dead && gt == 0) sh->stop_flag[slot] = 1;
            named_bar(3, CONSUMERS);
        }
        // closing barrier of the item: every store of the item precedes the count that publishes it
        dead = dead || (*(volatile int*)&sh->dead[g] != 0);
        if (dead && lane == 0) sh->stop_flag[slot] = 1;
        named_bar(3, CONSUMERS);
        if (release_a_after_close) release(0);
        const bool stop_now = *(volatile int*)&sh->stop_flag[slot] != 0;
        if (tid == 0 && done_ctr != nullptr && !stop_now) { __threadfence(); red_release(done_ctr, 1); }
        if (stop_now) {
            if (tid == 0) atomicExch(a.ctrl + 1, 1);
            break;
        }
    }
}

}  // namespace gleam
