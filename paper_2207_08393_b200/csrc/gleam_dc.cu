// Host side of the C ABI declared in include/gleam.h: argument validation, workspace layout and
// the sequence of kernel launches for each problem class.
//
//   readout-invariant mask, fft_rank 2 :  [z = R^H y table]  ->  fused row kernel (one pass)
//   readout-invariant mask, fft_rank 3 :  [z table]  ->  per chunk of readout slabs:
//                                         rows forward -> columns (mask, residual) -> rows inverse
//   full mask                           :  rows forward -> strided axes -> rows inverse on a
//                                         coil-volume workspace
//
// With a mask that does not depend on the readout index the readout transform commutes with the
// mask, so A^H(Ax - y) = S^H P^H M (M P S x - R^H y) with P over the phase-encode axes and R over
// the readout axis only; R^H y is needed at sampled positions alone.
#include "../../include/gleam.h"
#include "size_ops.cuh"
#include "dc_rowtile.cuh"
#include "dc_fused3d.cuh"
#include "dc_fused_entry.h"
#include "dc_entry.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <vector>

namespace gleam {

#define GLEAM_SIZE(N, A0, A1, A2, LR, B0, B1, B2, LC) extern const SizeOps size_ops_##N;
#include "sizes.def"
#undef GLEAM_SIZE

const PairOps* find_pair(int n1, int n2);     // kernels_pairs.cu

static const SizeOps* find_size(int n) {
    switch (n) {
#define GLEAM_SIZE(N, A0, A1, A2, LR, B0, B1, B2, LC) case N: return &size_ops_##N;
#include "sizes.def"
#undef GLEAM_SIZE
        default: return nullptr;
    }
}

// Ranks of the sampled phase-encode positions, in the order of the raw (half-shifted) k index q:
//   zidx[bt][q]  = rank of q among the sampled positions, or -1 where M[sh(q)] == 0
//   zlist[bt][r] = unshifted source position p = sh(q) of rank r;   zcount[bt] = number sampled.
// Block (chunk, bt) owns ZMAP_CHUNK consecutive q; it counts the sampled positions before its chunk
// by itself (no communication between blocks), then scans its own chunk.
#define ZMAP_THREADS 1024
#define ZMAP_PER_THREAD 2
#define ZMAP_CHUNK (ZMAP_THREADS * ZMAP_PER_THREAD)
#define ZMAP_TILE 8
#define ZMAP_MAX_RY 32
__global__ void __launch_bounds__(ZMAP_THREADS) zmap_kernel(const float* __restrict__ mask, int* __restrict__ zidx,
                                                            int* __restrict__ zlist, int* __restrict__ zcount,
                                                            float* __restrict__ m2c, int* __restrict__ zstart,
                                                            int* __restrict__ chunk_cnt, int count_only,
                                                            int n1, int n2, int rank, int ry) {
    __shared__ int warp_sum[ZMAP_THREADS / 32];
    __shared__ int base_sh;
    const int pe = (rank == 2) ? n2 : n1 * n2;
    const long long bt = blockIdx.y;
    const float* mk = mask + bt * pe;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q_begin = blockIdx.x * ZMAP_CHUNK;
    // Rank order.  rank 2: the raw k index.  rank 3: column tiles of ZMAP_TILE raw kz indices, inside
    // a tile by (raw ky, raw kz): the sampled entries that one tile of the column kernel needs are
    // then neighbours in the compact z table.  raw_of maps the scan position to the raw position.
    // ry > 0 (row-tile path): groups of equal ky mod ry, inside a group by (ky div ry, kz): the sampled
    // entries one block of the row-tile middle pass needs are contiguous; zstart[bt][k0] is the
    // first rank of group k0, zstart[bt][ry] the total.
    const bool tiled = (ry == 0) && (rank == 3) && (n2 % ZMAP_TILE == 0);
    const int per_k0 = (ry > 0) ? (n1 / ry) * n2 : 1;
    auto raw_of = [&](int q) -> int {
        if (ry > 0) {
            const int k0 = q / per_k0, rem = q - k0 * per_k0;
            return (k0 + ry * (rem / n2)) * n2 + rem % n2;
        }
        if (!tiled) return q;
        const int per_tile = n1 * ZMAP_TILE;
        const int tile = q / per_tile, rem = q - tile * per_tile;
        return (rem / ZMAP_TILE) * n2 + tile * ZMAP_TILE + rem % ZMAP_TILE;
    };
    auto src_of = [&](int q) -> int {            // unshifted source position of scan position q
        const int rq = raw_of(q);
        if (rank == 2) return shift_half(rq, n2);
        return shift_half(rq / n2, n1) * n2 + shift_half(rq % n2, n2);
    };
    // Two launches: the first (count_only) stores the number of sampled positions of every chunk,
    // the second adds up the chunks before its own and numbers its entries.
    const int nchunks = gridDim.x;
    if (count_only) {
        int c = 0;
#pragma unroll
        for (int e = 0; e < ZMAP_PER_THREAD; ++e) {
            const int q = q_begin + tid * ZMAP_PER_THREAD + e;
            c += (q < pe && mk[src_of(q)] != 0.f) ? 1 : 0;
        }
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0) warp_sum[warp] = c;
        __syncthreads();
        if (tid == 0) { int t = 0; for (int w = 0; w < ZMAP_THREADS / 32; ++w) t += warp_sum[w]; chunk_cnt[bt * nchunks + blockIdx.x] = t; }
        return;
    }
    if (tid == 0) { int t = 0; for (int w = 0; w < (int)blockIdx.x; ++w) t += chunk_cnt[bt * nchunks + w]; base_sh = t; }
    __syncthreads();
    const int base = base_sh;
    __syncthreads();
    // this chunk: each thread owns ZMAP_PER_THREAD consecutive q
    const int q0 = q_begin + tid * ZMAP_PER_THREAD;
    int src[ZMAP_PER_THREAD]; bool on[ZMAP_PER_THREAD]; int mine = 0;
#pragma unroll
    for (int e = 0; e < ZMAP_PER_THREAD; ++e) {
        const int q = q0 + e;
        src[e] = (q < pe) ? src_of(q) : 0;
        on[e] = (q < pe) && (mk[src[e]] != 0.f);
        mine += on[e] ? 1 : 0;
    }
    int incl = mine;                                         // inclusive scan inside the warp
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    int wbase = 0;
    for (int w = 0; w < warp; ++w) wbase += warp_sum[w];
    int r = base + wbase + incl - mine;
#pragma unroll
    for (int e = 0; e < ZMAP_PER_THREAD; ++e) {
        const int q = q0 + e;
        if (q >= pe) break;
        if (ry > 0 && q % per_k0 == 0) zstart[bt * (ZMAP_MAX_RY + 1) + q / per_k0] = r;
        if (on[e]) {
            const float mv = mk[src[e]];
            zidx[bt * pe + raw_of(q)] = r; zlist[bt * pe + r] = src[e]; m2c[bt * pe + r] = mv * mv; ++r;
        }
        else zidx[bt * pe + raw_of(q)] = -1;
    }
    if (q_begin + ZMAP_CHUNK >= pe && tid == ZMAP_THREADS - 1) {                 // last chunk, last thread: total
        zcount[bt] = r;
        if (ry > 0) zstart[bt * (ZMAP_MAX_RY + 1) + ry] = r;
    }
}

static inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

struct Layout {
    // geometry
    int B, C, T, Ts, rank, n0, n1, n2;
    long long V, units, images;
    bool separable;
    // workspace (byte offsets)
    uint64_t off_z, off_zidx, off_zlist, off_zcount, off_m2c, off_zstart, off_zchunk, off_W, total;
    int G;  // readout slabs per chunk (rank 3 separable)
    // fused persistent kernel of the separable 3-D path: control words first (at offset 0, the same
    // for forward and VJP calls, so that gleam_dc_check_status finds them), then the ring of R slabs
    bool fused;
    uint64_t off_ctrl, ctrl_bytes, off_ring;
    int R, L2, L3;
};

// Ring size and lags of the fused kernel, in slabs.  One block per SM is resident and a period of one slab has fewer
// items than there are SMs, so three to four slabs are in flight per pass and a dependency is only surely met after
// about four periods: P2 follows P1 by L2 = 4 periods, P3 by L3 = 8, and the ring holds R = 16 slabs (84 MB for 8
// coils of 320 x 256).  Measured per VJP call on the 320 x 320 x 256 volume: (8, 2, 4) 2.36 ms, (12, 3, 6) 2.04 ms,
// (16, 4, 8) 1.81 ms.  GLEAM_FUSED_RING="R,L2,L3" overrides (tuning aid, read once).
static void fused_ring(int* R, int* L2, int* L3) {
    static int v[3] = {0, 0, 0};
    if (v[0] == 0) {
        int r = 16, l2 = 4, l3 = 8;
        const char* e = getenv("GLEAM_FUSED_RING");
        if (e) { int a = 0, b = 0, c = 0; if (sscanf(e, "%d,%d,%d", &a, &b, &c) == 3 && a > c && c >= b && b >= 1 && a <= 64) { r = a; l2 = b; l3 = c; } }
        v[1] = l2; v[2] = l3; v[0] = r;
    }
    *R = v[0]; *L2 = v[1]; *L3 = v[2];
}
// The persistent kernel is opt-in: measured on the 320 x 320 x 256 volume it only draws level with the three
// whole-volume passes (1.81 ms against 1.77-1.93 ms per VJP call), so the default keeps those.  GLEAM_FUSED=1 in the environment
// or gleam_dc_set_fused(1) selects it; the choice changes the workspace layout, so it is made before
// gleam_dc_workspace_size.
static std::atomic<int> g_fused_on{-1};
static bool fused_enabled() {
    int v = g_fused_on.load(std::memory_order_relaxed);
    if (v < 0) { const char* e = getenv("GLEAM_FUSED"); v = (e && e[0] == '1') ? 1 : 0; g_fused_on.store(v); }
    return v == 1;
}

// Target size of the 3-D chunk workspace.  A chunk of about 48 MB would stay inside L2 between the
// three kernels of a chunk, but at their present speed the kernels are bound by instruction issue,
// not by bandwidth, and fewer, larger launches measure faster; the default therefore covers the
// whole volume up to 2 GB.  GLEAM_CHUNK_MB overrides it (tuning aid, read once).
static uint64_t chunk_target_bytes() {
    static uint64_t v = 0;
    if (v == 0) {
        const char* e = getenv("GLEAM_CHUNK_MB");
        long mb = e ? atol(e) : 0;
        v = (uint64_t)((mb > 0 && mb <= 65536) ? mb : 2048) << 20;
    }
    return v;
}

static int make_layout(const gleam_dims* d, bool with_y, Layout* L) {
    if (d->struct_version != GLEAM_DIMS_VERSION) return GLEAM_ERR_BAD_DIMS;
    if (d->batch < 1 || d->coils < 1 || d->frames < 1) return GLEAM_ERR_BAD_DIMS;
    if (d->fft_rank != 2 && d->fft_rank != 3) return GLEAM_ERR_BAD_DIMS;
    if (d->n[0] < 1 || d->n[1] < 1 || d->n[2] < 1) return GLEAM_ERR_BAD_DIMS;
    if (d->fft_rank == 2 && d->n[0] != 1) return GLEAM_ERR_BAD_DIMS;
    if (d->sens_has_frames != 0 && d->sens_has_frames != 1) return GLEAM_ERR_BAD_DIMS;
    if (d->mask_kind != GLEAM_MASK_FULL && d->mask_kind != GLEAM_MASK_READOUT_INVARIANT) return GLEAM_ERR_BAD_DIMS;
    for (int a = 3 - d->fft_rank; a < 3; ++a)
        if (!find_size(d->n[a])) return GLEAM_ERR_UNSUPPORTED_SIZE;
    L->B = d->batch; L->C = d->coils; L->T = d->frames; L->Ts = d->sens_has_frames ? d->frames : 1;
    L->rank = d->fft_rank; L->n0 = d->n[0]; L->n1 = d->n[1]; L->n2 = d->n[2];
    L->V = (long long)L->n0 * L->n1 * L->n2;
    L->images = (long long)L->B * L->T;
    L->units = L->images * L->C;
    if (L->V > (1ll << 40) || L->units * L->V > (1ll << 46)) return GLEAM_ERR_BAD_DIMS;
    if ((long long)L->n1 * L->n2 >= (1ll << 30) || L->images > 65535) return GLEAM_ERR_BAD_DIMS;   // rank map: 32-bit positions, grid.y
    if (L->images * L->n0 * L->n1 >= (1ll << 31)) return GLEAM_ERR_BAD_DIMS;   // row counters are 32-bit
    L->separable = d->mask_kind == GLEAM_MASK_READOUT_INVARIANT;
    uint64_t off = 0;
    L->off_z = L->off_zidx = L->off_zlist = L->off_zcount = L->off_m2c = L->off_zstart = L->off_zchunk = L->off_W = 0; L->G = 0;
    L->fused = false; L->off_ctrl = L->ctrl_bytes = L->off_ring = 0; L->R = L->L2 = L->L3 = 0;
    if (L->separable && L->rank == 3 && fused_enabled() && fused3d_supported(L->n1, L->n2) &&
        L->images * L->n0 < (1ll << 24)) {
        L->fused = true;
        fused_ring(&L->R, &L->L2, &L->L3);
        const long long nslabs = L->images * L->n0;
        if (L->R > nslabs + L->L3) L->R = (int)(nslabs + L->L3);      // never more slots than slabs in flight
        if (L->R <= L->L3) L->R = L->L3 + 1;
        L->off_ctrl = off; L->ctrl_bytes = (uint64_t)(64 + 3 * nslabs) * sizeof(int);
        off = align_up(off + L->ctrl_bytes, 256);
        L->off_ring = off; off = align_up(off + (uint64_t)L->R * L->C * L->n1 * L->n2 * sizeof(cf), 256);
    }
    if (L->separable) {
        const long long pe = (L->rank == 2) ? L->n2 : (long long)L->n1 * L->n2;
        if (with_y) {
            // compact z table, sized for the worst case (every position sampled), and the rank maps
            L->off_z = off; off = align_up(off + (uint64_t)L->units * L->V * sizeof(cf), 256);
            L->off_zidx = off; off = align_up(off + (uint64_t)L->images * pe * sizeof(int), 256);
            L->off_zlist = off; off = align_up(off + (uint64_t)L->images * pe * sizeof(int), 256);
            L->off_zcount = off; off = align_up(off + (uint64_t)L->images * sizeof(int), 256);
            L->off_m2c = off; off = align_up(off + (uint64_t)L->images * pe * sizeof(float), 256);
            L->off_zstart = off; off = align_up(off + (uint64_t)L->images * (ZMAP_MAX_RY + 1) * sizeof(int), 256);
            L->off_zchunk = off; off = align_up(off + (uint64_t)L->images * ((pe + ZMAP_CHUNK - 1) / ZMAP_CHUNK) * sizeof(int), 256);
        }
        if (L->rank == 3) {
            const uint64_t slab = (uint64_t)L->units * L->n1 * L->n2 * sizeof(cf);
            long long G = (long long)(chunk_target_bytes() / slab);
            if (G < 1) G = 1;
            if (G > L->n0) G = L->n0;
            L->G = (int)G;
            L->off_W = off; off = align_up(off + slab * (uint64_t)G, 256);
        }
    } else {
        L->off_W = off; off = align_up(off + (uint64_t)L->units * L->V * sizeof(cf), 256);
    }
    L->total = off;
    return GLEAM_OK;
}

static bool check_pointers_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("GLEAM_SKIP_POINTER_CHECK"); v = (e && e[0] == '1') ? 0 : 1; }
    return v == 1;
}

int check_device_ptr(const void* p) {
    if (!check_pointers_enabled()) return GLEAM_OK;
    cudaPointerAttributes at;
    cudaError_t e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) { cudaGetLastError(); return GLEAM_ERR_NOT_DEVICE_POINTER; }
    if (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) return GLEAM_ERR_NOT_DEVICE_POINTER;
    return GLEAM_OK;
}

static bool overlaps(const void* a, uint64_t na, const void* b, uint64_t nb) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

static inline float gsign(int n) { return ((n / 2) % 2) ? -1.f : 1.f; }

#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return GLEAM_ERR_CUDA; } while (0)

// ---- launch counter and optional per-kernel event timing (measurement aid) ----
static std::atomic<unsigned long long> g_launches{0};
static std::mutex g_prof_mutex;
static bool g_prof_on = false;
static std::vector<cudaEvent_t> g_prof_events;   // event i is recorded just before launch i
static std::vector<int> g_prof_class;            // kernel class of launch i, -1 = end-of-call marker
static size_t g_prof_used = 0;

cudaError_t prof_mark(int cls, cudaStream_t s) {
    if (cls >= 0) g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_prof_on) return cudaSuccess;
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (g_prof_used == g_prof_events.size()) {
        cudaEvent_t e;
        cudaError_t r = cudaEventCreate(&e);
        if (r != cudaSuccess) return r;
        g_prof_events.push_back(e);
        g_prof_class.push_back(cls);
    }
    g_prof_class[g_prof_used] = cls;
    return cudaEventRecord(g_prof_events[g_prof_used++], s);
}
#define LAUNCH(cls, call) do { CK(prof_mark((cls), s)); CK(call); } while (0)

bool dot_rows_supported(const gleam_dims* d) {
    if (!d || d->fft_rank != 2 || d->mask_kind != GLEAM_MASK_READOUT_INVARIANT) return false;
    const SizeOps* op2 = find_size(d->n[2]);
    return op2 && op2->row_is_warp_resident;
}

int run(const void* x, const void* y, const void* sens, const float* mask, float eta, void* out,
        const gleam_dims* d, int mode, double* dot_rows, bool check_only, int layout, const void* aty) {
    if (!d || !mask) return GLEAM_ERR_NULL_POINTER;
    if (aty && (y || mode != RUN_ALL)) return GLEAM_ERR_BAD_DIMS;      // the given A^H y stands in for y
    if (mode == RUN_PREPARE) {
        if (!y) return GLEAM_ERR_NULL_POINTER;
        x = nullptr; sens = nullptr; out = nullptr;
    } else if (!x || !sens || !out) {
        return GLEAM_ERR_NULL_POINTER;
    }
    if (mode == RUN_APPLY && !y) return GLEAM_ERR_NULL_POINTER;
    if (dot_rows && !dot_rows_supported(d)) return GLEAM_ERR_UNIMPLEMENTED;   // callers ask first
    Layout L;
    int rc = make_layout(d, y != nullptr, &L);
    if (rc != GLEAM_OK) return rc;
    if (L.total > 0 && !d->workspace) return GLEAM_ERR_NULL_POINTER;
    if (d->workspace_bytes < L.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)d->workspace & 255) != 0) return GLEAM_ERR_BAD_DIMS;

    const uint64_t img_b = (uint64_t)L.images * L.V * sizeof(cf);
    const uint64_t ksp_b = (uint64_t)L.units * L.V * sizeof(cf);
    const uint64_t sens_b = (uint64_t)L.B * L.C * L.Ts * L.V * sizeof(cf);
    const long long pe = (L.rank == 2) ? L.n2 : (long long)L.n1 * L.n2;
    const uint64_t mask_b = (uint64_t)L.images * (L.separable ? pe : L.V) * sizeof(float);
    const void* ptrs[7] = {x, y, sens, mask, out, d->workspace, aty};
    for (int i = 0; i < 7; ++i) {
        if (!ptrs[i]) continue;
        if (((uintptr_t)ptrs[i] & 15) != 0) return GLEAM_ERR_BAD_DIMS;   // 16-byte copies
        rc = check_device_ptr(ptrs[i]);
        if (rc != GLEAM_OK) return rc;
    }
    // aliasing: out may equal x exactly; nothing else may overlap an output or the workspace
    if (layout & ~(GLEAM_X_CHANNELS | GLEAM_OUT_CHANNELS)) return GLEAM_ERR_BAD_DIMS;
    if (mode != RUN_PREPARE) {
        if (out != x && overlaps(out, img_b, x, img_b)) return GLEAM_ERR_ALIAS;
        if (out == x && ((layout & GLEAM_X_CHANNELS) != 0) != ((layout & GLEAM_OUT_CHANNELS) != 0)) return GLEAM_ERR_ALIAS;
        if (overlaps(out, img_b, sens, sens_b) || overlaps(out, img_b, mask, mask_b)) return GLEAM_ERR_ALIAS;
        if (y && overlaps(out, img_b, y, ksp_b)) return GLEAM_ERR_ALIAS;
        if (aty && overlaps(out, img_b, aty, img_b)) return GLEAM_ERR_ALIAS;
    }
    if (L.total > 0) {
        const void* w = d->workspace;
        if ((mode != RUN_PREPARE && (overlaps(w, L.total, x, img_b) || overlaps(w, L.total, out, img_b) ||
                                     overlaps(w, L.total, sens, sens_b))) ||
            overlaps(w, L.total, mask, mask_b) || (y && overlaps(w, L.total, y, ksp_b)) ||
            (aty && overlaps(w, L.total, aty, img_b)))
            return GLEAM_ERR_ALIAS;
    }
    if (check_only) return GLEAM_OK;          // every argument check has passed; nothing is enqueued

    cudaStream_t s = (cudaStream_t)d->stream;
    char* ws = (char*)d->workspace;
    const SizeOps* op2 = find_size(L.n2);
    const SizeOps* op1 = find_size(L.n1);
    const SizeOps* op0 = (L.rank == 3) ? find_size(L.n0) : nullptr;

    RowArgs ra{};
    ra.x = (const cf*)x; ra.sens = (const cf*)sens; ra.out = (cf*)out; ra.eta = eta;
    ra.C = L.C; ra.T = L.T; ra.Ts = L.Ts; ra.RPB = L.n0 * L.n1;
    ra.x_planar = (layout & GLEAM_X_CHANNELS) ? 1 : 0; ra.out_planar = (layout & GLEAM_OUT_CHANNELS) ? 1 : 0;
    ra.plane = (long long)L.T * L.V;
    ra.aty = (const cf*)aty;
    ColArgs ca{};
    ca.C = L.C; ca.T = L.T; ca.rank = L.rank; ca.n0 = L.n0; ca.n1 = L.n1; ca.n2 = L.n2;

    if (L.separable) {
        cf* z = y ? (cf*)(ws + L.off_z) : nullptr;
        if (y) {
            // ranks of the sampled positions, then the z table: inverse transform of y along the
            // readout axis at the sampled positions only
            int* zidx = (int*)(ws + L.off_zidx);
            int* zlist = (int*)(ws + L.off_zlist);
            int* zcount = (int*)(ws + L.off_zcount);
            float* m2c = (float*)(ws + L.off_m2c);
            int* zstart = (int*)(ws + L.off_zstart);
            const PairOps* zpair = (L.rank == 3) ? find_pair(L.n1, L.n2) : nullptr;
            const int zry = (zpair && zpair->ry <= ZMAP_MAX_RY) ? zpair->ry : 0;
            int* zchunk = (int*)(ws + L.off_zchunk);
            const dim3 zgrid((unsigned)((pe + ZMAP_CHUNK - 1) / ZMAP_CHUNK), (unsigned)L.images);
            // rank 2 with a one-pass row kernel that counts the sampled positions itself: nothing
            // but the z table needs the ranks, and the kernel that writes it derives them per block
            const bool self_ranks = L.rank == 2 && op2->row_is_warp_resident && pe <= COLZ_SELF_MAX;
            if (mode != RUN_APPLY && !self_ranks) {      // RUN_APPLY: the tables of an earlier RUN_PREPARE are in the workspace
                CK(prof_mark(GLEAM_K_PREP_M2, s));
                if (zgrid.x > 1) {        // a table of one chunk needs no counts of earlier chunks
                    zmap_kernel<<<zgrid, ZMAP_THREADS, 0, s>>>(mask, zidx, zlist, zcount, m2c, zstart, zchunk, 1, L.n1, L.n2, L.rank, zry);
                    CK(cudaGetLastError());
                    CK(prof_mark(GLEAM_K_PREP_M2, s));
                }
                zmap_kernel<<<zgrid, ZMAP_THREADS, 0, s>>>(mask, zidx, zlist, zcount, m2c, zstart, zchunk, 0, L.n1, L.n2, L.rank, zry);
                CK(cudaGetLastError());
            }
            ca.zidx = zidx; ca.zlist = zlist; ca.zcount = zcount; ca.m2c = m2c; ca.zstart = zry ? zstart : nullptr;
            ra.zidx = zidx;
            ColArgs cz = ca;
            cz.y = (const cf*)y; cz.z = z; cz.mask = mask;
            if (self_ranks) { cz.zlist = nullptr; cz.zcount = nullptr; cz.zidx = nullptr; }
            cz.es = (int)pe; cz.nouter = L.units;
            const int nro = (L.rank == 2) ? L.n1 : L.n0;
            float g = gsign(nro) * gsign(L.n2) * (L.rank == 3 ? gsign(L.n1) : 1.f);
            cz.scale = g / sqrtf((float)nro * (float)pe);
            if (mode != RUN_APPLY) LAUNCH(GLEAM_K_COL_Z, ((L.rank == 2) ? op1 : op0)->col(COL_Z, cz, s));
        }
        if (mode == RUN_PREPARE) { CK(prof_mark(-1, s)); return GLEAM_OK; }
        if (L.rank == 2) {
            ra.mask = mask; ra.z = z; ra.rpb = L.n1; ra.row0 = 0; ra.nrows = L.images * L.n1;
            ra.dot_rows = dot_rows;
            LAUNCH(GLEAM_K_ROW_FUSED, op2->row(ROW_FUSED, ra, s));
        } else {
            if (L.fused && !y && !aty && layout == 0) {
                // one persistent kernel walks all slabs; its counters start from zero
                FusedArgs fa{};
                fa.x = (const cf*)x; fa.sens = (const cf*)sens; fa.out = (cf*)out; fa.W = (cf*)(ws + L.off_ring);
                fa.mask = mask; fa.zin = z; fa.zidx = ca.zidx; fa.m2c = ca.m2c; fa.zstart = ca.zstart;
                fa.ctrl = (int*)(ws + L.off_ctrl); fa.eta = eta; fa.scale2 = 1.0f / (float)pe;
                fa.C = L.C; fa.T = L.T; fa.Ts = L.Ts; fa.n0 = L.n0; fa.nslabs = (int)(L.images * L.n0);
                fa.R = L.R; fa.L2 = L.L2; fa.L3 = L.L3;
                fa.withhold = fused3d_withhold(); fa.limit_ns = fused3d_limit_ns();
                CK(cudaMemsetAsync(fa.ctrl, 0, L.ctrl_bytes, s));
                LAUNCH(GLEAM_K_FUSED3D, fused3d_launch(L.n1, fa, s));
                CK(prof_mark(-1, s));
                return GLEAM_OK;
            }
            cf* W = (cf*)(ws + L.off_W);
            const PairOps* pair = find_pair(L.n1, L.n2);
            for (int i0 = 0; i0 < L.n0; i0 += L.G) {
                const int g = (L.n0 - i0 < L.G) ? (L.n0 - i0) : L.G;
                if (pair) {
                    // row-tile kernels: every pass over the workspace is contiguous
                    TileArgs ta{};
                    ta.x = (const cf*)x; ta.sens = (const cf*)sens; ta.out = (cf*)out; ta.V = W; ta.mask = mask;
                    ta.zin = z; ta.zidx = ca.zidx; ta.m2c = ca.m2c; ta.zstart = ca.zstart; ta.eta = eta; ta.scale2 = 1.0f / (float)pe;
                    ta.C = L.C; ta.T = L.T; ta.Ts = L.Ts; ta.n0 = L.n0; ta.G = g; ta.i0_start = i0; ta.nunits = L.units;
                    ta.x_planar = ra.x_planar; ta.out_planar = ra.out_planar; ta.plane = ra.plane; ta.aty = ra.aty;
                    LAUNCH(GLEAM_K_ROW_FWD, pair->fwd(ta, L.images, s));
                    LAUNCH(GLEAM_K_COL_MID_SEP, pair->mid(ta, s));
                    LAUNCH(GLEAM_K_ROW_INV, pair->inv(ta, L.images, s));
                    continue;
                }
                ra.W = W; ra.rpb = g * L.n1; ra.row0 = i0 * L.n1; ra.nrows = L.images * ra.rpb;
                LAUNCH(GLEAM_K_ROW_FWD, op2->row(ROW_FWD, ra, s));
                ColArgs cm = ca;
                cm.W = W; cm.mask = mask; cm.scale2 = 1.0f / (float)pe; cm.zin = z; cm.es = L.n2; cm.nouter = L.units * g; cm.G = g; cm.i0_start = i0;
                LAUNCH(GLEAM_K_COL_MID_SEP, op1->col(COL_MID_SEP, cm, s));
                LAUNCH(GLEAM_K_ROW_INV, op2->row(ROW_INV, ra, s));
            }
        }
    } else {
        if (mode == RUN_PREPARE) return GLEAM_OK;      // a full mask has nothing to prepare
        cf* W = (cf*)(ws + L.off_W);
        ra.W = W; ra.rpb = L.n0 * L.n1; ra.row0 = 0; ra.nrows = L.images * ra.rpb;
        LAUNCH(GLEAM_K_ROW_FWD, op2->row(ROW_FWD, ra, s));
        float g = gsign(L.n2) * gsign(L.n1) * (L.rank == 3 ? gsign(L.n0) : 1.f);
        const double ntot = (L.rank == 3) ? (double)L.V : (double)L.n1 * L.n2;
        ColArgs cm = ca;
        cm.W = W; cm.y = (const cf*)y; cm.mask = mask;
        cm.scale = g / (float)sqrt(ntot); cm.scale2 = (float)(1.0 / ntot);
        if (L.rank == 2) {
            cm.es = L.n2; cm.nouter = L.units;
            LAUNCH(GLEAM_K_COL_MID_FULL, op1->col(COL_MID_FULL, cm, s));
        } else {
            ColArgs c1 = ca;
            c1.W = W; c1.es = L.n2; c1.nouter = L.units * L.n0;
            LAUNCH(GLEAM_K_COL_FWD, op1->col(COL_FWD, c1, s));
            cm.es = L.n1 * L.n2; cm.nouter = L.units;
            LAUNCH(GLEAM_K_COL_MID_FULL, op0->col(COL_MID_FULL, cm, s));
            LAUNCH(GLEAM_K_COL_INV, op1->col(COL_INV, c1, s));
        }
        LAUNCH(GLEAM_K_ROW_INV, op2->row(ROW_INV, ra, s));
    }
    CK(prof_mark(-1, s));
    return GLEAM_OK;
}


// ---- gradients of Eq. 3 with respect to the measurements and the step size ----
// <g, a> per batch example, double accumulation in a fixed order: block partial sums, then one block per example.
#define GRAD_THREADS 256
#define GRAD_MAX_BLOCKS 512
__global__ void __launch_bounds__(GRAD_THREADS) grad_eta_partial_kernel(const cf* __restrict__ g, const cf* __restrict__ x,
                                                                        const cf* __restrict__ t, long long ne,
                                                                        double* __restrict__ part) {
    // t = x - A^H(Ax - y)  (the step with eta = 1), so A^H(Ax - y) = x - t
    __shared__ double sh[GRAD_THREADS];
    const long long base = (long long)blockIdx.y * ne;
    double acc = 0.0;
    for (long long i = (long long)blockIdx.x * GRAD_THREADS + threadIdx.x; i < ne; i += (long long)gridDim.x * GRAD_THREADS) {
        const cf gv = g[base + i], xv = x[base + i], tv = t[base + i];
        acc += (double)gv.x * ((double)xv.x - (double)tv.x) + (double)gv.y * ((double)xv.y - (double)tv.y);
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int o = GRAD_THREADS / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) part[(long long)blockIdx.y * gridDim.x + blockIdx.x] = sh[0];
}
__global__ void grad_eta_final_kernel(const double* __restrict__ part, int nblocks, double* __restrict__ grad_eta) {
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < nblocks; ++i) s += part[(long long)blockIdx.x * nblocks + i];
        grad_eta[blockIdx.x] = -s;
    }
}


// ---- complex l1 loss between an image and a reference (training loss of the paper's networks) ----
// loss = mean |x - r|; grad = (x - r) / |x - r| / N (zero where x = r).  Block partial sums in double, summed
// by one thread in block order: deterministic.
__global__ void __launch_bounds__(GRAD_THREADS) l1_partial_kernel(const cf* __restrict__ x, const cf* __restrict__ r, cf* __restrict__ grad,
                                                                  long long ne, int B, int x_planar, int g_planar, long long plane,
                                                                  float inv_n, double* __restrict__ part) {
    __shared__ double sh[GRAD_THREADS];
    double acc = 0.0;
    const long long n = ne * B;
    for (long long i = (long long)blockIdx.x * GRAD_THREADS + threadIdx.x; i < n; i += (long long)gridDim.x * GRAD_THREADS) {
        const int b = (int)(i / ne);
        const cf xv = load_image(x, i, x_planar, b, plane), rv = r[i];
        const float dx = xv.x - rv.x, dy = xv.y - rv.y;
        const float m = sqrtf(dx * dx + dy * dy);
        acc += (double)m;
        if (grad) {
            const float s = m > 0.f ? inv_n / m : 0.f;
            store_image(grad, i, make_float2(dx * s, dy * s), g_planar, b, plane);
        }
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int o = GRAD_THREADS / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) part[blockIdx.x] = sh[0];
}
__global__ void l1_final_kernel(const double* __restrict__ part, int nblocks, double inv_n, double* __restrict__ loss) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < nblocks; ++i) s += part[i];
        *loss = s * inv_n;
    }
}


// ---- FP32 peak probe (measurement aid): independent FMA chains, no memory traffic ----
__global__ void __launch_bounds__(256) fma_peak_kernel(float* sink, int iters, float a, float b) {
    float v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = (float)(threadIdx.x + i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = fmaf(v[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += v[i];
    if (s == 12345.678f) sink[0] = s;              // never true: keeps the chains alive
}

struct GradLayout { uint64_t dc_bytes, off_t, off_part, off_W, total; long long ne; int nblocks; };
static int grad_layout(const gleam_dims* d, GradLayout* G) {
    Layout L;
    int rc = make_layout(d, true, &L);
    if (rc != GLEAM_OK) return rc;
    G->dc_bytes = align_up(L.total, 256);
    G->ne = (long long)L.T * L.V;
    long long nb = (G->ne + GRAD_THREADS * 8 - 1) / (GRAD_THREADS * 8);
    G->nblocks = (int)(nb < 1 ? 1 : (nb > GRAD_MAX_BLOCKS ? GRAD_MAX_BLOCKS : nb));
    uint64_t off = G->dc_bytes;
    G->off_t = off; off = align_up(off + (uint64_t)L.images * L.V * sizeof(cf), 256);
    G->off_part = off; off = align_up(off + (uint64_t)L.B * G->nblocks * sizeof(double), 256);
    const uint64_t wbytes = (uint64_t)L.units * L.V * sizeof(cf);          // coil-volume workspace of the measurement gradient
    G->off_W = 0;
    G->total = off > wbytes ? off : align_up(wbytes, 256);
    return GLEAM_OK;
}

}  // namespace gleam

extern "C" {

GLEAM_API int gleam_dc_forward(const void* x, const void* y, const void* sens, const float* mask, float eta,
                     void* out, const gleam_dims* dims) {
    if (!y) return GLEAM_ERR_NULL_POINTER;
    return gleam::run(x, y, sens, mask, eta, out, dims);
}

GLEAM_API int gleam_dc_vjp(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_in,
                 const gleam_dims* dims) {
    return gleam::run(grad_out, nullptr, sens, mask, eta, grad_in, dims);
}

GLEAM_API int gleam_dc_forward_layout(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                      void* out, const gleam_dims* dims, uint32_t layout) {
    if (!y) return GLEAM_ERR_NULL_POINTER;
    return gleam::run(x, y, sens, mask, eta, out, dims, gleam::RUN_ALL, nullptr, false, (int)layout);
}

GLEAM_API int gleam_dc_vjp_layout(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_in,
                                  const gleam_dims* dims, uint32_t layout) {
    return gleam::run(grad_out, nullptr, sens, mask, eta, grad_in, dims, gleam::RUN_ALL, nullptr, false, (int)layout);
}

GLEAM_API int gleam_dc_adjoint(const void* y, const void* sens, const float* mask, void* out, const gleam_dims* dims) {
    if (!dims || !y || !sens || !mask || !out) return GLEAM_ERR_NULL_POINTER;
    if (((uintptr_t)out & 15) != 0) return GLEAM_ERR_BAD_DIMS;
    int rc = gleam::check_device_ptr(out);
    if (rc != GLEAM_OK) return rc;
    // all argument checks of the step itself, before the output is cleared
    rc = gleam::run(out, y, sens, mask, 1.0f, out, dims, gleam::RUN_ALL, nullptr, true);
    if (rc != GLEAM_OK) return rc;
    const uint64_t img_b = (uint64_t)dims->batch * dims->frames * dims->n[0] * dims->n[1] * dims->n[2] * sizeof(gleam::cf);
    if (cudaMemsetAsync(out, 0, img_b, (cudaStream_t)dims->stream) != cudaSuccess) return GLEAM_ERR_CUDA;
    return gleam::run(out, y, sens, mask, 1.0f, out, dims);     // 0 - 1 * A^H (A 0 - y), in place
}

GLEAM_API int gleam_dc_forward_aty(const void* x, const void* aty, const void* sens, const float* mask, float eta,
                                   void* out, const gleam_dims* dims) {
    if (!aty) return GLEAM_ERR_NULL_POINTER;
    return gleam::run(x, nullptr, sens, mask, eta, out, dims, gleam::RUN_ALL, nullptr, false, 0, aty);
}

GLEAM_API int gleam_dc_prepare(const void* y, const float* mask, const gleam_dims* dims) {
    return gleam::run(nullptr, y, nullptr, mask, 0.f, nullptr, dims, gleam::RUN_PREPARE);
}

GLEAM_API int gleam_dc_forward_prepared(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                        void* out, const gleam_dims* dims) {
    return gleam::run(x, y, sens, mask, eta, out, dims, gleam::RUN_APPLY);
}

GLEAM_API int gleam_dc_workspace_size(const gleam_dims* dims, uint64_t* bytes) {
    if (!dims || !bytes) return GLEAM_ERR_NULL_POINTER;
    gleam::Layout L;
    int rc = gleam::make_layout(dims, true, &L);
    if (rc != GLEAM_OK) return rc;
    *bytes = L.total;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_check_status(const gleam_dims* dims) {
    if (!dims) return GLEAM_ERR_NULL_POINTER;
    gleam::Layout L;
    int rc = gleam::make_layout(dims, true, &L);
    if (rc != GLEAM_OK) return rc;
    if (cudaStreamSynchronize((cudaStream_t)dims->stream) != cudaSuccess) return GLEAM_ERR_CUDA;
    if (!L.fused) return GLEAM_OK;                  // no kernel of this problem class waits on another block
    if (!dims->workspace) return GLEAM_ERR_NULL_POINTER;
    if (dims->workspace_bytes < L.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    int word = 0;
    if (cudaMemcpy(&word, (const char*)dims->workspace + L.off_ctrl + sizeof(int), sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return GLEAM_ERR_CUDA;
    return word == 0 ? GLEAM_OK : GLEAM_ERR_TIMEOUT;
}

GLEAM_API int gleam_dc_fused_wait_stats(const gleam_dims* dims, uint64_t* ns_and_counts, int32_t n_kinds) {
    if (!dims || !ns_and_counts) return GLEAM_ERR_NULL_POINTER;
    gleam::Layout L;
    int rc = gleam::make_layout(dims, true, &L);
    if (rc != GLEAM_OK) return rc;
    for (int i = 0; i < 2 * n_kinds; ++i) ns_and_counts[i] = 0;
    if (!L.fused) return GLEAM_OK;
    if (!dims->workspace || dims->workspace_bytes < L.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (cudaStreamSynchronize((cudaStream_t)dims->stream) != cudaSuccess) return GLEAM_ERR_CUDA;
    uint64_t w[10];
    if (cudaMemcpy(w, (const char*)dims->workspace + L.off_ctrl + 8 * sizeof(int), sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess)
        return GLEAM_ERR_CUDA;
    for (int i = 0; i < 2 * (n_kinds < 5 ? n_kinds : 5); ++i) ns_and_counts[i] = w[i];
    return GLEAM_OK;
}

GLEAM_API int32_t gleam_dc_rowtile_split(int32_t n1, int32_t n2) {
    const gleam::PairOps* p = gleam::find_pair(n1, n2);
    return p ? p->ry : 0;
}

GLEAM_API void gleam_dc_set_fused(int32_t on) { gleam::g_fused_on.store(on ? 1 : 0); }

GLEAM_API void gleam_dc_debug_fused(int32_t withhold_item, uint64_t wait_limit_ns) {
    gleam::fused3d_set_debug(withhold_item, wait_limit_ns);
}

GLEAM_API int gleam_measure_fp32_peak(void* scratch4, void* stream, double* tflops) {
    if (!scratch4 || !tflops) return GLEAM_ERR_NULL_POINTER;
    int rc = gleam::check_device_ptr(scratch4);
    if (rc != GLEAM_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GLEAM_ERR_CUDA;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return GLEAM_ERR_CUDA;
    const int iters = 1 << 14, blocks = sms * 8;
    double best = 0.0;
    for (int rep = 0; rep < 5; ++rep) {
        cudaEventRecord(e0, s);
        gleam::fma_peak_kernel<<<blocks, 256, 0, s>>>((float*)scratch4, iters, 0.999f, 0.001f);
        cudaEventRecord(e1, s);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaEventDestroy(e0); cudaEventDestroy(e1); return GLEAM_ERR_CUDA; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double tf = 2.0 * 16.0 * iters * 256.0 * blocks / (ms * 1e-3) / 1e12;
        if (rep > 0 && tf > best) best = tf;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    *tflops = best;
    return GLEAM_OK;
}

GLEAM_API uint64_t gleam_l1_loss_workspace_size(void) { return GRAD_MAX_BLOCKS * sizeof(double); }

GLEAM_API int gleam_l1_loss(const void* x, const void* ref, double* loss, void* grad, const gleam_dims* dims, uint32_t layout) {
    using namespace gleam;
    if (!dims || !x || !ref || !loss) return GLEAM_ERR_NULL_POINTER;
    Layout L;
    int rc = make_layout(dims, false, &L);
    if (rc != GLEAM_OK) return rc;
    if (layout & ~(GLEAM_X_CHANNELS | GLEAM_OUT_CHANNELS)) return GLEAM_ERR_BAD_DIMS;
    if (!dims->workspace) return GLEAM_ERR_NULL_POINTER;
    if (dims->workspace_bytes < gleam_l1_loss_workspace_size()) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)x & 7) || ((uintptr_t)ref & 7) || ((uintptr_t)loss & 7) || ((uintptr_t)grad & 7) || ((uintptr_t)dims->workspace & 255)) return GLEAM_ERR_BAD_DIMS;
    const void* ptrs[5] = {x, ref, loss, grad, dims->workspace};
    for (int i = 0; i < 5; ++i) if (ptrs[i] && (rc = check_device_ptr(ptrs[i])) != GLEAM_OK) return rc;
    const uint64_t img_b = (uint64_t)L.images * L.V * sizeof(cf);
    if (grad && grad != x && (overlaps(grad, img_b, x, img_b) || overlaps(grad, img_b, ref, img_b))) return GLEAM_ERR_ALIAS;
    if (grad == x && ((layout & GLEAM_X_CHANNELS) != 0) != ((layout & GLEAM_OUT_CHANNELS) != 0)) return GLEAM_ERR_ALIAS;
    if (overlaps(dims->workspace, gleam_l1_loss_workspace_size(), x, img_b) || overlaps(dims->workspace, gleam_l1_loss_workspace_size(), ref, img_b) ||
        (grad && overlaps(dims->workspace, gleam_l1_loss_workspace_size(), grad, img_b)) || overlaps(loss, 8, x, img_b) ||
        (grad && overlaps(loss, 8, grad, img_b)))
        return GLEAM_ERR_ALIAS;
    const long long ne = (long long)L.T * L.V, n = ne * L.B;
    long long nb = (n + GRAD_THREADS * 8 - 1) / (GRAD_THREADS * 8);
    const int nblocks = (int)(nb < 1 ? 1 : (nb > GRAD_MAX_BLOCKS ? GRAD_MAX_BLOCKS : nb));
    cudaStream_t s = (cudaStream_t)dims->stream;
    double* part = (double*)dims->workspace;
    CK(prof_mark(GLEAM_K_CG_VEC, s));
    l1_partial_kernel<<<nblocks, GRAD_THREADS, 0, s>>>((const cf*)x, (const cf*)ref, (cf*)grad, ne, L.B, (layout & GLEAM_X_CHANNELS) ? 1 : 0,
                                                       (layout & GLEAM_OUT_CHANNELS) ? 1 : 0, ne, (float)(1.0 / (double)n), part);
    CK(cudaGetLastError());
    CK(prof_mark(GLEAM_K_CG_VEC, s));
    l1_final_kernel<<<1, 32, 0, s>>>(part, nblocks, 1.0 / (double)n, loss);
    CK(cudaGetLastError());
    CK(prof_mark(-1, s));
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_grad_workspace_size(const gleam_dims* dims, uint64_t* bytes) {
    if (!dims || !bytes) return GLEAM_ERR_NULL_POINTER;
    gleam::GradLayout G;
    int rc = gleam::grad_layout(dims, &G);
    if (rc != GLEAM_OK) return rc;
    *bytes = G.total;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_grad_eta(const void* grad_out, const void* x, const void* y, const void* sens, const float* mask,
                                double* grad_eta, const gleam_dims* dims) {
    using namespace gleam;
    if (!dims || !grad_out || !x || !y || !sens || !mask || !grad_eta) return GLEAM_ERR_NULL_POINTER;
    GradLayout G;
    int rc = grad_layout(dims, &G);
    if (rc != GLEAM_OK) return rc;
    if (!dims->workspace) return GLEAM_ERR_NULL_POINTER;
    if (dims->workspace_bytes < G.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)grad_out & 15) != 0 || ((uintptr_t)grad_eta & 7) != 0 || ((uintptr_t)dims->workspace & 255) != 0) return GLEAM_ERR_BAD_DIMS;
    if ((rc = check_device_ptr(grad_out)) != GLEAM_OK || (rc = check_device_ptr(grad_eta)) != GLEAM_OK) return rc;
    char* ws = (char*)dims->workspace;
    const uint64_t img_b = (uint64_t)dims->batch * G.ne * sizeof(cf);
    if (overlaps(ws, G.total, grad_out, img_b) || overlaps(ws, G.total, grad_eta, (uint64_t)dims->batch * 8) ||
        overlaps(grad_eta, (uint64_t)dims->batch * 8, grad_out, img_b) || overlaps(grad_eta, (uint64_t)dims->batch * 8, x, img_b))
        return GLEAM_ERR_ALIAS;
    gleam_dims d = *dims;
    d.workspace = ws; d.workspace_bytes = G.dc_bytes;
    cf* t = (cf*)(ws + G.off_t);
    rc = run(x, y, sens, mask, 1.0f, t, &d, RUN_ALL, nullptr, true);       // every argument check before anything is enqueued
    if (rc != GLEAM_OK) return rc;
    rc = run(x, y, sens, mask, 1.0f, t, &d);                               // t = x - A^H (A x - y)
    if (rc != GLEAM_OK) return rc;
    cudaStream_t s = (cudaStream_t)dims->stream;
    double* part = (double*)(ws + G.off_part);
    if (prof_mark(GLEAM_K_CG_VEC, s) != cudaSuccess) return GLEAM_ERR_CUDA;
    grad_eta_partial_kernel<<<dim3((unsigned)G.nblocks, (unsigned)dims->batch), GRAD_THREADS, 0, s>>>((const cf*)grad_out, (const cf*)x, t, G.ne, part);
    if (cudaGetLastError() != cudaSuccess) return GLEAM_ERR_CUDA;
    if (prof_mark(GLEAM_K_CG_VEC, s) != cudaSuccess) return GLEAM_ERR_CUDA;
    grad_eta_final_kernel<<<(unsigned)dims->batch, 32, 0, s>>>(part, G.nblocks, grad_eta);
    if (cudaGetLastError() != cudaSuccess) return GLEAM_ERR_CUDA;
    if (prof_mark(-1, s) != cudaSuccess) return GLEAM_ERR_CUDA;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_grad_y(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_y,
                              const gleam_dims* dims) {
    using namespace gleam;
    if (!dims || !grad_out || !sens || !mask || !grad_y) return GLEAM_ERR_NULL_POINTER;
    Layout L;
    int rc = make_layout(dims, false, &L);
    if (rc != GLEAM_OK) return rc;
    GradLayout G;
    if ((rc = grad_layout(dims, &G)) != GLEAM_OK) return rc;
    if (!dims->workspace) return GLEAM_ERR_NULL_POINTER;
    if (dims->workspace_bytes < G.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)dims->workspace & 255) != 0) return GLEAM_ERR_BAD_DIMS;
    const void* ptrs[5] = {grad_out, sens, mask, grad_y, dims->workspace};
    for (int i = 0; i < 5; ++i) {
        if (((uintptr_t)ptrs[i] & 15) != 0) return GLEAM_ERR_BAD_DIMS;
        if ((rc = check_device_ptr(ptrs[i])) != GLEAM_OK) return rc;
    }
    const uint64_t img_b = (uint64_t)L.images * L.V * sizeof(cf), ksp_b = (uint64_t)L.units * L.V * sizeof(cf);
    const uint64_t sens_b = (uint64_t)L.B * L.C * L.Ts * L.V * sizeof(cf);
    const long long pe = (L.rank == 2) ? L.n2 : (long long)L.n1 * L.n2;
    const uint64_t mask_b = (uint64_t)L.images * (L.separable ? pe : L.V) * sizeof(float);
    if (overlaps(grad_y, ksp_b, grad_out, img_b) || overlaps(grad_y, ksp_b, sens, sens_b) || overlaps(grad_y, ksp_b, mask, mask_b) ||
        overlaps(dims->workspace, G.total, grad_y, ksp_b) || overlaps(dims->workspace, G.total, grad_out, img_b) ||
        overlaps(dims->workspace, G.total, sens, sens_b) || overlaps(dims->workspace, G.total, mask, mask_b))
        return GLEAM_ERR_ALIAS;
    cudaStream_t s = (cudaStream_t)dims->stream;
    cf* W = (cf*)((char*)dims->workspace + G.off_W);
    const SizeOps* op2 = find_size(L.n2);
    const SizeOps* op1 = find_size(L.n1);
    const SizeOps* op0 = (L.rank == 3) ? find_size(L.n0) : nullptr;
    RowArgs ra{};
    ra.x = (const cf*)grad_out; ra.sens = (const cf*)sens; ra.W = W; ra.eta = 0.f;
    ra.C = L.C; ra.T = L.T; ra.Ts = L.Ts; ra.RPB = L.n0 * L.n1; ra.rpb = ra.RPB; ra.row0 = 0; ra.nrows = L.images * ra.rpb;
    LAUNCH(GLEAM_K_ROW_FWD, op2->row(ROW_FWD, ra, s));
    ColArgs ca{};
    ca.C = L.C; ca.T = L.T; ca.rank = L.rank; ca.n0 = L.n0; ca.n1 = L.n1; ca.n2 = L.n2; ca.W = W;
    const float gs = gsign(L.n2) * gsign(L.n1) * (L.rank == 3 ? gsign(L.n0) : 1.f);
    const double ntot = (L.rank == 3) ? (double)L.V : (double)L.n1 * L.n2;
    ColArgs cy = ca;
    cy.mask = mask; cy.ky_out = (cf*)grad_y; cy.mask_pe = L.separable ? (int)pe : 0;
    cy.scale = eta * gs / (float)sqrt(ntot);
    if (L.rank == 2) {
        cy.es = L.n2; cy.nouter = L.units;
        LAUNCH(GLEAM_K_COL_FWD, op1->col(COL_GRADY, cy, s));
    } else {
        ColArgs c1 = ca;
        c1.es = L.n2; c1.nouter = L.units * L.n0;
        LAUNCH(GLEAM_K_COL_FWD, op1->col(COL_FWD, c1, s));
        cy.es = L.n1 * L.n2; cy.nouter = L.units;
        LAUNCH(GLEAM_K_COL_FWD, op0->col(COL_GRADY, cy, s));
    }
    CK(prof_mark(-1, s));
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_length_supported(int32_t n) {
    return gleam::find_size(n) ? GLEAM_OK : GLEAM_ERR_UNSUPPORTED_SIZE;
}

GLEAM_API const char* gleam_status_string(int status) {
    switch (status) {
        case GLEAM_OK: return "ok";
        case GLEAM_ERR_NULL_POINTER: return "null pointer argument";
        case GLEAM_ERR_BAD_DIMS: return "inconsistent or misaligned dims";
        case GLEAM_ERR_UNSUPPORTED_SIZE: return "transform length not supported";
        case GLEAM_ERR_NOT_DEVICE_POINTER: return "argument is not a device pointer";
        case GLEAM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GLEAM_ERR_ALIAS: return "arguments overlap";
        case GLEAM_ERR_CUDA: return "CUDA runtime error";
        case GLEAM_ERR_UNIMPLEMENTED: return "not implemented";
        case GLEAM_ERR_TIMEOUT: return "device wait timed out";
        default: return "unknown status";
    }
}

GLEAM_API int gleam_version(void) { return GLEAM_VERSION; }

// ---- fixed scratch for callers that cannot allocate device memory ----
// One array per GPU that loads this library, resident until the process exits.
#define GLEAM_STATIC_SCRATCH_BYTES (64ull << 20)
static __device__ __align__(256) unsigned char g_static_scratch[GLEAM_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not an address the GPU can
// use, so the device address is looked up once per device (with that device current) and cached.
static int static_scratch_address(void** out) {
    enum { MAX_DEVICES = 64 };
    static void* cache[MAX_DEVICES] = {nullptr};
    static std::mutex mtx;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return GLEAM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mtx);
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return GLEAM_ERR_CUDA; }
        cache[dev] = p;
    }
    *out = cache[dev];
    return GLEAM_OK;
}

GLEAM_API uint64_t gleam_dc_static_scratch_bytes(void) { return GLEAM_STATIC_SCRATCH_BYTES; }

GLEAM_API int gleam_dc_forward_static(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                      void* out, const gleam_dims* dims) {
    if (!dims || !y) return GLEAM_ERR_NULL_POINTER;
    gleam::Layout L;
    int rc = gleam::make_layout(dims, true, &L);
    if (rc != GLEAM_OK) return rc;
    if (L.total > GLEAM_STATIC_SCRATCH_BYTES) return GLEAM_ERR_WORKSPACE_TOO_SMALL;   // problem too large for the fixed scratch
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != GLEAM_OK) return rc;
    gleam_dims d = *dims;
    d.workspace = scratch;
    d.workspace_bytes = GLEAM_STATIC_SCRATCH_BYTES;
    // Every scratch element that the kernels read is written earlier in the same call, so nothing
    // has to be cleared between calls even though the array keeps the previous call's contents.
    return gleam::run(x, y, sens, mask, eta, out, &d);
}

GLEAM_API uint64_t gleam_dc_launch_count(void) { return gleam::g_launches.load(); }

GLEAM_API int gleam_dc_profile_begin(void) {
    std::lock_guard<std::mutex> lock(gleam::g_prof_mutex);
    gleam::g_prof_on = true;
    gleam::g_prof_used = 0;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_profile_end(float* ms, uint32_t* launches, int32_t n_classes) {
    using namespace gleam;
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    g_prof_on = false;
    if (!ms || !launches) return GLEAM_ERR_NULL_POINTER;
    for (int i = 0; i < n_classes; ++i) { ms[i] = 0.f; launches[i] = 0; }
    if (g_prof_used == 0) return GLEAM_OK;
    if (cudaEventSynchronize(g_prof_events[g_prof_used - 1]) != cudaSuccess) return GLEAM_ERR_CUDA;
    for (size_t i = 0; i + 1 < g_prof_used; ++i) {
        const int cls = g_prof_class[i];
        if (cls < 0 || cls >= n_classes) continue;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, g_prof_events[i], g_prof_events[i + 1]) != cudaSuccess) return GLEAM_ERR_CUDA;
        ms[cls] += t;
        launches[cls] += 1;
    }
    g_prof_used = 0;
    return GLEAM_OK;
}

static int host_arena_layout(const gleam_dims* d, uint64_t off[7], uint64_t sz[6]) {
    gleam::Layout L;
    int rc = gleam::make_layout(d, true, &L);
    if (rc != GLEAM_OK) return rc;
    const long long pe = (L.rank == 2) ? L.n2 : (long long)L.n1 * L.n2;
    sz[0] = (uint64_t)L.images * L.V * 8;                                   // x / grad_out
    sz[1] = (uint64_t)L.units * L.V * 8;                                    // y
    sz[2] = (uint64_t)L.B * L.C * L.Ts * L.V * 8;                           // sens
    sz[3] = (uint64_t)L.images * (L.separable ? pe : L.V) * 4;              // mask
    sz[4] = sz[0];                                                          // out
    sz[5] = L.total;                                                        // workspace
    uint64_t o = 0;
    for (int i = 0; i < 6; ++i) { off[i] = o; o = gleam::align_up(o + sz[i], 256); }
    off[6] = o;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_host_arena_size(const gleam_dims* dims, uint64_t* bytes) {
    if (!dims || !bytes) return GLEAM_ERR_NULL_POINTER;
    uint64_t off[7], sz[6];
    int rc = host_arena_layout(dims, off, sz);
    if (rc != GLEAM_OK) return rc;
    *bytes = off[6];
    return GLEAM_OK;
}

static int run_host(const void* x, const void* y, const void* sens, const float* mask, float eta, void* out,
                    const gleam_dims* dims, void* arena, uint64_t arena_bytes) {
    if (!dims || !x || !sens || !mask || !out || !arena) return GLEAM_ERR_NULL_POINTER;
    if (((uintptr_t)arena & 255) != 0) return GLEAM_ERR_BAD_DIMS;
    uint64_t off[7], sz[6];
    int rc = host_arena_layout(dims, off, sz);
    if (rc != GLEAM_OK) return rc;
    if (arena_bytes < off[6]) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    char* a = (char*)arena;
    cudaStream_t s = (cudaStream_t)dims->stream;
    gleam_dims d = *dims;
    d.workspace = a + off[5];
    d.workspace_bytes = sz[5];
    // argument checks on the staged device pointers come before the first copy is enqueued
    rc = gleam::run(a + off[0], y ? a + off[1] : nullptr, a + off[2], (const float*)(a + off[3]), eta, a + off[4], &d,
                    gleam::RUN_ALL, nullptr, true);
    if (rc != GLEAM_OK) return rc;
    const void* src[4] = {x, y, sens, mask};
    for (int i = 0; i < 4; ++i) {
        if (!src[i]) continue;
        if (cudaMemcpyAsync(a + off[i], src[i], sz[i], cudaMemcpyHostToDevice, s) != cudaSuccess) return GLEAM_ERR_CUDA;
    }
    rc = gleam::run(a + off[0], y ? a + off[1] : nullptr, a + off[2], (const float*)(a + off[3]), eta, a + off[4], &d);
    if (rc != GLEAM_OK) return rc;
    if (cudaMemcpyAsync(out, a + off[4], sz[4], cudaMemcpyDeviceToHost, s) != cudaSuccess) return GLEAM_ERR_CUDA;
    return GLEAM_OK;
}

GLEAM_API int gleam_dc_forward_host(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                    void* out, const gleam_dims* dims, void* arena, uint64_t arena_bytes) {
    if (!y) return GLEAM_ERR_NULL_POINTER;
    return run_host(x, y, sens, mask, eta, out, dims, arena, arena_bytes);
}

GLEAM_API int gleam_dc_vjp_host(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_in,
                                const gleam_dims* dims, void* arena, uint64_t arena_bytes) {
    return run_host(grad_out, nullptr, sens, mask, eta, grad_in, dims, arena, arena_bytes);
}

}  // extern "C"
