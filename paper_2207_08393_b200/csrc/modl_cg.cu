// MoDL data-consistency step (Eq. 7, second line):  out = (A^H A + mu I)^{-1} (A^H y + mu z)
// by a fixed number of conjugate-gradient steps, and its vector-Jacobian product with respect to z.
//
// The normal operator is the data-consistency VJP path of this library with eta = -1/mu:
//     q = p + (1/mu) A^H A p = H p / mu,          H = A^H A + mu I,
// so the factor mu moves into the scalars (alpha = <r,r> / (mu <p,q>),  r -= alpha mu q) and no
// operator kernel changes.  The right-hand side A^H y is the forward call on a zero image with
// eta = 1.  What remains are image-sized vector updates with inner products per batch example:
//
//     cg_init : b = A^H y + mu z  (VJP: b = mu g);  r = p = b;  x = 0;  partial sums of <b,b>
//     cg_dot  : partial sums of Re <p,q>
//     cg_step : alpha = rr / (mu pq);  x += alpha p;  r -= alpha mu q;  partial sums of <r,r>
//     cg_dir  : beta = rr' / rr;  p = r + beta p
//
// Where the operator is the one-pass 2-D kernel, that kernel also stores Re<p_row, q_row> of every
// image row it writes (it holds both in registers at its update step) and cg_dot is not launched.
//
// Inner products: every thread accumulates in double precision, a block reduces in a fixed order
// and stores one partial sum; the kernel that needs the scalar adds the partial sums of its example
// in a fixed order at its start (every block the same sum).  Producer and consumer are different
// launches on one stream: no atomics, no fences, no block waits for another one, and the result
// does not depend on the order in which blocks run.  <r,r> alternates between two partial-sum
// arrays (step parity) because cg_dir needs the old and the new value.
#include "dc_entry.h"

#include <cmath>
#include <cstdint>

namespace gleam {

constexpr int CG_THREADS = 256;
constexpr int CG_MAX_BLOCKS = 592;          // partial sums per example (4 blocks per SM on 148 SMs)

struct CgArgs {
    const float4* z;         // z (forward) or grad_out (VJP), two complex values per element
    const float4* q;         // A^H y at cg_init, H p / mu afterwards
    float4* r; float4* p; float4* x;
    double* part_rr;         // (2, B, CG_MAX_BLOCKS): <r,r> partial sums of even / odd steps
    double* part_pq;         // (B, CG_MAX_BLOCKS): <p,q> partial sums written by cg_dot
    const double* dot_rows;  // (B, rows_per_example): Re<p,q> per image row from the operator, or null
    int rows_per_example;
    long long ne2;           // float4 elements per example
    float mu;
    int parity;              // step k & 1: part_rr[parity] holds <r_k, r_k>
};

// Sum of v over the block in a fixed order; the same value in every thread.
__device__ __forceinline__ double block_sum(double v) {
    __shared__ double warp_sum[CG_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    __syncthreads();                                    // earlier readers of warp_sum are done
    if (lane == 0) warp_sum[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < CG_THREADS / 32; ++w) t += warp_sum[w];
    return t;
}

// Sum of n values written by an earlier launch (fixed order: thread t takes t, t + 256, ...).
__device__ __forceinline__ double array_sum(const double* v, int n) {
    double t = 0.0;
    for (int i = threadIdx.x; i < n; i += CG_THREADS) t += __ldcg(v + i);
    return block_sum(t);
}

__device__ __forceinline__ double* rr_slot(const CgArgs& a, int which) {
    return a.part_rr + ((size_t)which * gridDim.y + blockIdx.y) * CG_MAX_BLOCKS;
}

__device__ __forceinline__ double norm2(float4 v) {
    return (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
}

template <bool HAS_Q>
__global__ void __launch_bounds__(CG_THREADS) cg_init_kernel(const CgArgs a) {
    const long long base = (long long)blockIdx.y * a.ne2;
    double acc = 0.0;
    for (long long i = (long long)blockIdx.x * CG_THREADS + threadIdx.x; i < a.ne2; i += (long long)gridDim.x * CG_THREADS) {
        const float4 zv = a.z[base + i];
        float4 b = make_float4(a.mu * zv.x, a.mu * zv.y, a.mu * zv.z, a.mu * zv.w);
        if (HAS_Q) {
            const float4 qv = a.q[base + i];
            b = make_float4(fmaf(a.mu, zv.x, qv.x), fmaf(a.mu, zv.y, qv.y), fmaf(a.mu, zv.z, qv.z), fmaf(a.mu, zv.w, qv.w));
        }
        a.r[base + i] = b;
        a.p[base + i] = b;
        a.x[base + i] = make_float4(0.f, 0.f, 0.f, 0.f);
        acc += norm2(b);
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) rr_slot(a, 0)[blockIdx.x] = acc;
}

__global__ void __launch_bounds__(CG_THREADS) cg_dot_kernel(const CgArgs a) {
    const long long base = (long long)blockIdx.y * a.ne2;
    double acc = 0.0;
    for (long long i = (long long)blockIdx.x * CG_THREADS + threadIdx.x; i < a.ne2; i += (long long)gridDim.x * CG_THREADS) {
        const float4 pv = a.p[base + i], qv = a.q[base + i];
        acc += (double)pv.x * qv.x + (double)pv.y * qv.y + (double)pv.z * qv.z + (double)pv.w * qv.w;
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) a.part_pq[(size_t)blockIdx.y * CG_MAX_BLOCKS + blockIdx.x] = acc;
}

template <bool FROM_ROWS>
__global__ void __launch_bounds__(CG_THREADS) cg_step_kernel(const CgArgs a) {
    const long long base = (long long)blockIdx.y * a.ne2;
    const double rr = array_sum(rr_slot(a, a.parity), (int)gridDim.x);
    const double pq = FROM_ROWS ? array_sum(a.dot_rows + (size_t)blockIdx.y * a.rows_per_example, a.rows_per_example)
                                : array_sum(a.part_pq + (size_t)blockIdx.y * CG_MAX_BLOCKS, (int)gridDim.x);
    // an example whose residual is exactly zero stays as it is
    const double alpha = (rr > 0.0 && pq > 0.0) ? rr / ((double)a.mu * pq) : 0.0;
    const float af = (float)alpha, amu = (float)(alpha * (double)a.mu);
    double acc = 0.0;
    for (long long i = (long long)blockIdx.x * CG_THREADS + threadIdx.x; i < a.ne2; i += (long long)gridDim.x * CG_THREADS) {
        const float4 pv = a.p[base + i], qv = a.q[base + i];
        float4 xv = a.x[base + i], rv = a.r[base + i];
        xv = make_float4(fmaf(af, pv.x, xv.x), fmaf(af, pv.y, xv.y), fmaf(af, pv.z, xv.z), fmaf(af, pv.w, xv.w));
        rv = make_float4(fmaf(-amu, qv.x, rv.x), fmaf(-amu, qv.y, rv.y), fmaf(-amu, qv.z, rv.z), fmaf(-amu, qv.w, rv.w));
        a.x[base + i] = xv;
        a.r[base + i] = rv;
        acc += norm2(rv);
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) rr_slot(a, a.parity ^ 1)[blockIdx.x] = acc;
}

__global__ void __launch_bounds__(CG_THREADS) cg_dir_kernel(const CgArgs a) {
    const long long base = (long long)blockIdx.y * a.ne2;
    const double rr = array_sum(rr_slot(a, a.parity), (int)gridDim.x);
    const double rr_new = array_sum(rr_slot(a, a.parity ^ 1), (int)gridDim.x);
    const float beta = (rr > 0.0) ? (float)(rr_new / rr) : 0.f;
    for (long long i = (long long)blockIdx.x * CG_THREADS + threadIdx.x; i < a.ne2; i += (long long)gridDim.x * CG_THREADS) {
        const float4 rv = a.r[base + i], pv = a.p[base + i];
        a.p[base + i] = make_float4(fmaf(beta, pv.x, rv.x), fmaf(beta, pv.y, rv.y), fmaf(beta, pv.z, rv.z), fmaf(beta, pv.w, rv.w));
    }
}

static inline uint64_t up256(uint64_t v) { return (v + 255) / 256 * 256; }

struct CgLayout {
    uint64_t dc_bytes, img_bytes, off_q, off_r, off_p, off_rr, off_pq, off_rows, total;
    long long ne2;
    int B;
};

static int cg_layout(const gleam_dims* d, CgLayout* L) {
    if (!d) return GLEAM_ERR_NULL_POINTER;
    uint64_t dc = 0;
    const int rc = gleam_dc_workspace_size(d, &dc);          // validates dims; sized for the forward call
    if (rc != GLEAM_OK) return rc;
    const long long V = (long long)d->n[0] * d->n[1] * d->n[2];
    const long long ne = (long long)d->frames * V;            // complex values per example (even: V is even)
    L->B = d->batch;
    L->ne2 = ne / 2;
    L->dc_bytes = up256(dc);
    L->img_bytes = (uint64_t)d->batch * (uint64_t)ne * 8u;
    uint64_t off = L->dc_bytes;
    L->off_q = off; off = up256(off + L->img_bytes);
    L->off_r = off; off = up256(off + L->img_bytes);
    L->off_p = off; off = up256(off + L->img_bytes);
    L->off_rr = off; off = up256(off + 2u * (uint64_t)d->batch * CG_MAX_BLOCKS * sizeof(double));
    L->off_pq = off; off = up256(off + (uint64_t)d->batch * CG_MAX_BLOCKS * sizeof(double));
    L->off_rows = off; off = up256(off + (uint64_t)d->batch * d->frames * d->n[1] * sizeof(double));
    L->total = off;
    return GLEAM_OK;
}

static bool overlap(const void* a, uint64_t na, const void* b, uint64_t nb) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

#define CGCK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return GLEAM_ERR_CUDA; } while (0)
#define CGRUN(call) do { const int rc_ = (call); if (rc_ != GLEAM_OK) return rc_; } while (0)

// z: image (forward) or cotangent (VJP, y == nullptr)
static int modl_cg(const void* z, const void* y, const void* sens, const float* mask, float mu, int n_iter,
                   void* out, const gleam_dims* d) {
    if (!d || !z || !sens || !mask || !out) return GLEAM_ERR_NULL_POINTER;
    if (!(mu > 0.f) || !std::isfinite(mu) || n_iter < 0 || n_iter > 1000) return GLEAM_ERR_BAD_DIMS;
    CgLayout L;
    CGRUN(cg_layout(d, &L));
    if (!d->workspace) return GLEAM_ERR_NULL_POINTER;
    if (d->workspace_bytes < L.total) return GLEAM_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)d->workspace & 255) != 0) return GLEAM_ERR_BAD_DIMS;
    if ((((uintptr_t)z) & 15) != 0 || (((uintptr_t)out) & 15) != 0) return GLEAM_ERR_BAD_DIMS;
    CGRUN(check_device_ptr(z));
    CGRUN(check_device_ptr(out));
    CGRUN(check_device_ptr(d->workspace));
    // out may be z itself; nothing else may overlap the output or the workspace
    if (out != z && overlap(out, L.img_bytes, z, L.img_bytes)) return GLEAM_ERR_ALIAS;
    const uint64_t V = (uint64_t)d->n[0] * d->n[1] * d->n[2];
    const uint64_t ksp_bytes = L.img_bytes * (uint64_t)d->coils;
    const uint64_t sens_bytes = (uint64_t)d->batch * d->coils * (d->sens_has_frames ? d->frames : 1) * V * 8u;
    const uint64_t pe = (d->fft_rank == 2) ? (uint64_t)d->n[2] : (uint64_t)d->n[1] * d->n[2];
    const uint64_t mask_bytes = (uint64_t)d->batch * d->frames * (d->mask_kind == GLEAM_MASK_FULL ? V : pe) * 4u;
    if (overlap(d->workspace, L.total, z, L.img_bytes) || overlap(d->workspace, L.total, out, L.img_bytes) ||
        overlap(d->workspace, L.total, sens, sens_bytes) || overlap(d->workspace, L.total, mask, mask_bytes) ||
        (y && overlap(d->workspace, L.total, y, ksp_bytes)))
        return GLEAM_ERR_ALIAS;
    if (overlap(out, L.img_bytes, sens, sens_bytes) || overlap(out, L.img_bytes, mask, mask_bytes) ||
        (y && overlap(out, L.img_bytes, y, ksp_bytes)))
        return GLEAM_ERR_ALIAS;

    cudaStream_t s = (cudaStream_t)d->stream;
    char* ws = (char*)d->workspace;
    gleam_dims dd = *d;
    dd.workspace_bytes = L.dc_bytes;
    CgArgs a{};
    a.z = (const float4*)z; a.q = (const float4*)(ws + L.off_q);
    a.r = (float4*)(ws + L.off_r); a.p = (float4*)(ws + L.off_p); a.x = (float4*)out;
    a.part_rr = (double*)(ws + L.off_rr); a.part_pq = (double*)(ws + L.off_pq);
    a.ne2 = L.ne2; a.mu = mu; a.parity = 0;
    long long nb = (L.ne2 + (long long)CG_THREADS * 4 - 1) / ((long long)CG_THREADS * 4);
    if (nb < 1) nb = 1;
    if (nb > CG_MAX_BLOCKS) nb = CG_MAX_BLOCKS;
    const dim3 grid((unsigned)nb, (unsigned)L.B);
    // the one-pass 2-D operator kernel delivers <p,q> per image row
    const bool from_rows = dot_rows_supported(d);
    double* dot_rows = from_rows ? (double*)(ws + L.off_rows) : nullptr;
    a.dot_rows = dot_rows; a.rows_per_example = d->frames * d->n[1];

    // the operator's own argument checks (y, sens, mask) before anything is enqueued
    CGRUN(run(ws + L.off_r, y, sens, mask, 1.0f, ws + L.off_q, &dd, RUN_ALL, nullptr, true));
    if (y) {
        // A^H y: the forward call on a zero image with eta = 1
        CGCK(cudaMemsetAsync(ws + L.off_r, 0, L.img_bytes, s));
        CGRUN(run(ws + L.off_r, y, sens, mask, 1.0f, ws + L.off_q, &dd));
        CGCK(prof_mark(GLEAM_K_CG_VEC, s));
        cg_init_kernel<true><<<grid, CG_THREADS, 0, s>>>(a);
    } else {
        CGCK(prof_mark(GLEAM_K_CG_VEC, s));
        cg_init_kernel<false><<<grid, CG_THREADS, 0, s>>>(a);
    }
    CGCK(cudaGetLastError());
    for (int k = 0; k < n_iter; ++k) {
        a.parity = k & 1;
        CGRUN(run(a.p, nullptr, sens, mask, -1.0f / mu, ws + L.off_q, &dd, RUN_ALL, dot_rows));     // q = H p / mu
        if (from_rows) {
            CGCK(prof_mark(GLEAM_K_CG_VEC, s));
            cg_step_kernel<true><<<grid, CG_THREADS, 0, s>>>(a);
            CGCK(cudaGetLastError());
        } else {
            CGCK(prof_mark(GLEAM_K_CG_VEC, s));
            cg_dot_kernel<<<grid, CG_THREADS, 0, s>>>(a);
            CGCK(cudaGetLastError());
            CGCK(prof_mark(GLEAM_K_CG_VEC, s));
            cg_step_kernel<false><<<grid, CG_THREADS, 0, s>>>(a);
            CGCK(cudaGetLastError());
        }
        if (k + 1 < n_iter) {
            CGCK(prof_mark(GLEAM_K_CG_VEC, s));
            cg_dir_kernel<<<grid, CG_THREADS, 0, s>>>(a);
            CGCK(cudaGetLastError());
        }
    }
    CGCK(prof_mark(-1, s));
    return GLEAM_OK;
}

}  // namespace gleam

extern "C" {

GLEAM_API int gleam_modl_cg_forward(const void* z, const void* y, const void* sens, const float* mask, float mu,
                                    int32_t n_iter, void* out, const gleam_dims* dims) {
    if (!y) return GLEAM_ERR_NULL_POINTER;
    return gleam::modl_cg(z, y, sens, mask, mu, n_iter, out, dims);
}

GLEAM_API int gleam_modl_cg_vjp(const void* grad_out, const void* sens, const float* mask, float mu,
                                int32_t n_iter, void* grad_z, const gleam_dims* dims) {
    return gleam::modl_cg(grad_out, nullptr, sens, mask, mu, n_iter, grad_z, dims);
}

GLEAM_API int gleam_modl_cg_workspace_size(const gleam_dims* dims, uint64_t* bytes) {
    if (!dims || !bytes) return GLEAM_ERR_NULL_POINTER;
    gleam::CgLayout L;
    const int rc = gleam::cg_layout(dims, &L);
    if (rc != GLEAM_OK) return rc;
    *bytes = L.total;
    return GLEAM_OK;
}

}  // extern "C"
