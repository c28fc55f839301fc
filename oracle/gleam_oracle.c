/*
 * CPU oracle for the multi-coil SENSE data-consistency step  (TEST INFRASTRUCTURE).
 *
 * This file is test infrastructure only.  It is a slow, double-precision, obviously-correct
 * evaluation of the definitions in the GLEAM paper (arXiv 2207.08393).  It shares no code,
 * header, table or constant generator with the CUDA library, and the CUDA library never calls it.
 *
 *   Sensing model (Eq. 1):          y = Omega F S x + eps
 *   Forward operator (after Eq. 2): A = Omega F S ,  A^H its Hermitian transpose
 *   Data-consistency step (Eq. 3):  DC(x) = x - 2t A^H (A x - y)         (eta := 2t)
 *   Its vector-Jacobian product:    J^H g = g - eta A^H A g              (J = I - eta A^H A)
 *
 * Conventions the paper leaves open ("F is the Fourier transform matrix") and that are fixed
 * here:  F is the centred, orthonormal DFT over the trailing fft_rank spatial axes,
 *
 *      X[k] = N^(-1/2) * sum_n x[n] * exp(-2 pi i (k - o)(n - o) / N),    o = floor(N / 2),
 *
 * applied separably along every transformed axis; F^H uses +2 pi i.  Omega is a real diagonal
 * weight (normally 0/1) and is applied literally once in A and once in A^H:
 *      r_c = M .* (M .* F(S_c .* x) - y_c).
 *
 * Layout (row-major, last index fastest):
 *      x, out : (B, T, n0, n1, n2)           complex
 *      y      : (B, C, T, n0, n1, n2)        complex
 *      sens   : (B, C, n0, n1, n2)  or  (B, C, T, n0, n1, n2)   (sens_has_frames)
 *      mask   : mask_kind 0: (B, T, n0, n1, n2) real
 *               mask_kind 1: readout-invariant; fft_rank 2 -> (B, T, n2),  fft_rank 3 -> (B, T, n1, n2)
 * n0 = 1 when fft_rank == 2.  The frame axis T is never transformed.
 *
 * Inputs are single precision (the arrays the GPU sees), promoted to double; outputs are double.
 *
 * The MoDL model inversion of Eq. 7 by conjugate gradients is further down (oracle_modl_cg); its
 * pins are in tests/test_oracle_modl.py (closed form for A^H A = I, dense solve, Krylov-space
 * minimiser for the truncated iteration).
 *
 * Further down: the gradients of the step with respect to eta and y (oracle_dc_grad_eta,
 * oracle_dc_grad_y) and the bridge to the learned prior (two-channel layout, complex l1 loss); their
 * pins are in tests/test_oracle_bridge.py (dense-matrix brute force, exact difference quotients of
 * oracle_dc, an independent library routine for the layout, closed forms and central differences
 * for the loss).
 *
 * Pins (tests/test_oracle_pins.py): brute-force DFT, closed-form spectra of deltas and
 * constants, Parseval, adjoint identity, Hermitian/PSD normal operator, A^H A = I for a full mask
 * and unit-norm sensitivities, affine structure, an independent library FFT.
 */
#include <complex.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef double complex zc;

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_MEM (-2)

static const double TWO_PI = 6.283185307179586476925286766559;

/* ------------------------------------------------------------------------------------------
 * 1-D transforms
 * ---------------------------------------------------------------------------------------- */

/* The definition itself, by direct summation.  sign = -1: F (image -> k-space); +1: F^H.
 * The phase index (k-o)(n-o) is reduced modulo N in integers so that the argument of exp stays
 * in [0, 2 pi). */
void oracle_dft_naive_1d(const zc* in, zc* out, int64_t N, int sign)
{
    const int64_t o = N / 2;
    const double scale = 1.0 / sqrt((double)N);
    for (int64_t k = 0; k < N; ++k) {
        zc acc = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            int64_t p = ((k - o) * (n - o)) % N;
            if (p < 0) p += N;
            const double ang = sign * TWO_PI * (double)p / (double)N;
            acc += in[n] * (cos(ang) + I * sin(ang));
        }
        out[k] = acc * scale;
    }
}

/* Raw (uncentred, unscaled) DFT of a strided sequence: halve while the length is even
 * (decimation in time), evaluate the odd remainder by direct summation.
 * tw[j] = exp(sign 2 pi i j / N_top); at this level the root of unity is tw[tws]. */
static void fft_rec(const zc* in, int64_t stride, zc* out, int64_t n, const zc* tw, int64_t tws)
{
    if (n == 1) { out[0] = in[0]; return; }
    if (n % 2 != 0) {
        for (int64_t k = 0; k < n; ++k) {
            zc acc = 0.0;
            for (int64_t j = 0; j < n; ++j) acc += in[j * stride] * tw[((j * k) % n) * tws];
            out[k] = acc;
        }
        return;
    }
    const int64_t h = n / 2;
    fft_rec(in, 2 * stride, out, h, tw, 2 * tws);
    fft_rec(in + stride, 2 * stride, out + h, h, tw, 2 * tws);
    for (int64_t k = 0; k < h; ++k) {
        const zc e = out[k];
        const zc t = tw[k * tws] * out[k + h];
        out[k] = e + t;
        out[k + h] = e - t;
    }
}

/* Centred orthonormal transform: ifftshift -> raw FFT -> fftshift -> 1/sqrt(N).
 * Lengths up to 32 go through the direct sum.  work must hold 2 N entries, tw N entries
 * (tw[j] = exp(sign 2 pi i j / N)). */
static void fft_centered_line(const zc* in, zc* out, int64_t N, int sign, zc* work, const zc* tw)
{
    if (N <= 32) { oracle_dft_naive_1d(in, out, N, sign); return; }
    const int64_t o = N / 2;
    zc* a = work;
    zc* b = work + N;
    for (int64_t j = 0; j < N; ++j) a[j] = in[(j + o) % N];
    fft_rec(a, 1, b, N, tw, 1);
    const double scale = 1.0 / sqrt((double)N);
    for (int64_t j = 0; j < N; ++j) out[(j + o) % N] = b[j] * scale;
}

static zc* make_twiddles(int64_t N, int sign)
{
    zc* tw = (zc*)malloc(sizeof(zc) * (size_t)N);
    if (!tw) return NULL;
    for (int64_t j = 0; j < N; ++j) {
        const double ang = sign * TWO_PI * (double)j / (double)N;
        tw[j] = cos(ang) + I * sin(ang);
    }
    return tw;
}

int oracle_fft_centered_1d(const zc* in, zc* out, int64_t N, int sign)
{
    if (N < 1 || (sign != 1 && sign != -1)) return ORACLE_ERR_ARG;
    zc* work = (zc*)malloc(sizeof(zc) * (size_t)(2 * N));
    zc* tw = make_twiddles(N, sign);
    if (!work || !tw) { free(work); free(tw); return ORACLE_ERR_MEM; }
    fft_centered_line(in, out, N, sign, work, tw);
    free(work); free(tw);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * N-D transform over the trailing `rank` axes of `outer` volumes of shape n[0..2], in place.
 * ---------------------------------------------------------------------------------------- */
static int fft_centered_volume(zc* data, const int64_t n[3], int rank, int sign)
{
    const int64_t V = n[0] * n[1] * n[2];
    for (int ax = 3 - rank; ax < 3; ++ax) {
        const int64_t N = n[ax];
        if (N == 1) continue;
        int64_t stride = 1;
        for (int a = ax + 1; a < 3; ++a) stride *= n[a];
        const int64_t nlines = V / N;
        zc* tw = make_twiddles(N, sign);
        zc* buf = (zc*)malloc(sizeof(zc) * (size_t)(4 * N));
        if (!tw || !buf) { free(tw); free(buf); return ORACLE_ERR_MEM; }
        for (int64_t l = 0; l < nlines; ++l) {
            /* line l: all indices except axis ax */
            const int64_t inner = l % stride;
            const int64_t outerl = l / stride;
            zc* base = data + outerl * stride * N + inner;
            zc* li = buf;
            zc* lo = buf + N;
            for (int64_t j = 0; j < N; ++j) li[j] = base[j * stride];
            fft_centered_line(li, lo, N, sign, buf + 2 * N, tw);
            for (int64_t j = 0; j < N; ++j) base[j * stride] = lo[j];
        }
        free(tw); free(buf);
    }
    return ORACLE_OK;
}

/* Public: centred orthonormal DFT over the trailing `rank` axes of `outer` stacked volumes. */
int oracle_fftn_centered(zc* data, int64_t outer, const int64_t n[3], int rank, int sign, int nthreads)
{
    if (rank < 1 || rank > 3 || outer < 0) return ORACLE_ERR_ARG;
    const int64_t V = n[0] * n[1] * n[2];
    int rc = ORACLE_OK;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < outer; ++u) {
        const int r = fft_centered_volume(data + u * V, n, rank, sign);
        if (r != ORACLE_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc = r;
        }
    }
    return rc;
}

/* The definition in N-D by direct summation along each axis (tiny inputs only). */
int oracle_dftn_naive(zc* data, int64_t outer, const int64_t n[3], int rank, int sign)
{
    if (rank < 1 || rank > 3) return ORACLE_ERR_ARG;
    const int64_t V = n[0] * n[1] * n[2];
    for (int64_t u = 0; u < outer; ++u) {
        zc* vol = data + u * V;
        for (int ax = 3 - rank; ax < 3; ++ax) {
            const int64_t N = n[ax];
            int64_t stride = 1;
            for (int a = ax + 1; a < 3; ++a) stride *= n[a];
            zc* li = (zc*)malloc(sizeof(zc) * (size_t)(2 * N));
            if (!li) return ORACLE_ERR_MEM;
            zc* lo = li + N;
            for (int64_t l = 0; l < V / N; ++l) {
                zc* base = vol + (l / stride) * stride * N + (l % stride);
                for (int64_t j = 0; j < N; ++j) li[j] = base[j * stride];
                oracle_dft_naive_1d(li, lo, N, sign);
                for (int64_t j = 0; j < N; ++j) base[j * stride] = lo[j];
            }
            free(li);
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * The operators.  `dims` = {B, C, T, fft_rank, n0, n1, n2, sens_has_frames, mask_kind}.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int64_t B, C, T;
    int rank;
    int64_t n[3];
    int sens_has_frames;
    int mask_kind;
    int64_t V;
} odims;

static int parse_dims(const int64_t* d, odims* o)
{
    o->B = d[0]; o->C = d[1]; o->T = d[2]; o->rank = (int)d[3];
    o->n[0] = d[4]; o->n[1] = d[5]; o->n[2] = d[6];
    o->sens_has_frames = (int)d[7]; o->mask_kind = (int)d[8];
    if (o->B < 1 || o->C < 1 || o->T < 1) return ORACLE_ERR_ARG;
    if (o->rank != 2 && o->rank != 3) return ORACLE_ERR_ARG;
    if (o->n[0] < 1 || o->n[1] < 1 || o->n[2] < 1) return ORACLE_ERR_ARG;
    if (o->rank == 2 && o->n[0] != 1) return ORACLE_ERR_ARG;
    if (o->mask_kind != 0 && o->mask_kind != 1) return ORACLE_ERR_ARG;
    o->V = o->n[0] * o->n[1] * o->n[2];
    return ORACLE_OK;
}

/* Omega at voxel p of example b, frame t (p = flat index into (n0,n1,n2)). */
static inline double mask_at(const float* mask, const odims* o, int64_t b, int64_t t, int64_t p)
{
    if (o->mask_kind == 0) return (double)mask[(b * o->T + t) * o->V + p];
    /* readout-invariant: depends on the phase-encode indices only */
    if (o->rank == 2) return (double)mask[(b * o->T + t) * o->n[2] + (p % o->n[2])];
    const int64_t pe = o->n[1] * o->n[2];
    return (double)mask[(b * o->T + t) * pe + (p % pe)];
}

static inline const float* sens_ptr(const float* sens, const odims* o, int64_t b, int64_t c, int64_t t)
{
    const int64_t idx = o->sens_has_frames ? ((b * o->C + c) * o->T + t) : (b * o->C + c);
    return sens + 2 * idx * o->V;
}

/* k = A x  (Eq. 1 without noise):  k[b,c,t] = M .* F(S_c .* x).   k: (B,C,T,V) double complex. */
int oracle_apply_A(const float* x, const float* sens, const float* mask, const int64_t* dims,
                   zc* k, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK) return ORACLE_ERR_ARG;
    int rc = ORACLE_OK;
    const int64_t units = o.B * o.C * o.T;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < units; ++u) {
        const int64_t t = u % o.T, c = (u / o.T) % o.C, b = u / (o.T * o.C);
        const float* xs = x + 2 * (b * o.T + t) * o.V;
        const float* ss = sens_ptr(sens, &o, b, c, t);
        zc* ku = k + u * o.V;
        for (int64_t p = 0; p < o.V; ++p) {
            const zc xv = (double)xs[2 * p] + I * (double)xs[2 * p + 1];
            const zc sv = (double)ss[2 * p] + I * (double)ss[2 * p + 1];
            ku[p] = sv * xv;
        }
        const int r = fft_centered_volume(ku, o.n, o.rank, -1);
        if (r != ORACLE_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc = r;
        }
        for (int64_t p = 0; p < o.V; ++p) ku[p] *= mask_at(mask, &o, b, t, p);
    }
    return rc;
}

/* img = A^H k:  img[b,t] = sum_c conj(S_c) .* F^H (M .* k_c).   k is overwritten (scratch). */
int oracle_apply_AH(zc* k, const float* sens, const float* mask, const int64_t* dims,
                    zc* img, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK) return ORACLE_ERR_ARG;
    int rc = ORACLE_OK;
    const int64_t units = o.B * o.C * o.T;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < units; ++u) {
        const int64_t t = u % o.T, c = (u / o.T) % o.C, b = u / (o.T * o.C);
        const float* ss = sens_ptr(sens, &o, b, c, t);
        zc* ku = k + u * o.V;
        for (int64_t p = 0; p < o.V; ++p) ku[p] *= mask_at(mask, &o, b, t, p);
        const int r = fft_centered_volume(ku, o.n, o.rank, +1);
        if (r != ORACLE_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc = r;
        }
        for (int64_t p = 0; p < o.V; ++p) {
            const zc sv = (double)ss[2 * p] + I * (double)ss[2 * p + 1];
            ku[p] = conj(sv) * ku[p];
        }
    }
    /* coil sum in coil order (fixed order: result independent of the thread count) */
    for (int64_t b = 0; b < o.B; ++b)
        for (int64_t t = 0; t < o.T; ++t) {
            zc* dst = img + (b * o.T + t) * o.V;
            for (int64_t p = 0; p < o.V; ++p) dst[p] = 0.0;
            for (int64_t c = 0; c < o.C; ++c) {
                const zc* src = k + ((b * o.C + c) * o.T + t) * o.V;
                for (int64_t p = 0; p < o.V; ++p) dst[p] += src[p];
            }
        }
    return rc;
}

/* Eq. 3 with eta = 2t:   out = x - eta * A^H (A x - y).
 * y == NULL evaluates the vector-Jacobian product  out = x - eta * A^H A x  (x is then the
 * incoming cotangent).  Steps, in the order of the definition:
 *   1. c_c = S_c .* x          2. k_c = F c_c            3. r_c = M .* (M .* k_c - y_c)
 *   4. a = sum_c conj(S_c) .* F^H r_c                    5. out = x - eta a
 */
int oracle_dc(const float* x, const float* y, const float* sens, const float* mask, double eta,
              const int64_t* dims, zc* out, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK) return ORACLE_ERR_ARG;
    if (!x || !sens || !mask || !out) return ORACLE_ERR_ARG;
    zc* contrib = (zc*)malloc(sizeof(zc) * (size_t)(o.C * o.V));
    if (!contrib) return ORACLE_ERR_MEM;
    int rc = ORACLE_OK;
    if (nthreads < 1) nthreads = 1;
    for (int64_t b = 0; b < o.B; ++b)
        for (int64_t t = 0; t < o.T; ++t) {
            const float* xs = x + 2 * (b * o.T + t) * o.V;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
#endif
            for (int64_t c = 0; c < o.C; ++c) {
                const float* ss = sens_ptr(sens, &o, b, c, t);
                zc* w = contrib + c * o.V;
                /* 1 */
                for (int64_t p = 0; p < o.V; ++p) {
                    const zc xv = (double)xs[2 * p] + I * (double)xs[2 * p + 1];
                    const zc sv = (double)ss[2 * p] + I * (double)ss[2 * p + 1];
                    w[p] = sv * xv;
                }
                /* 2 */
                int r = fft_centered_volume(w, o.n, o.rank, -1);
                /* 3 */
                const float* ys = y ? y + 2 * ((b * o.C + c) * o.T + t) * o.V : NULL;
                for (int64_t p = 0; p < o.V; ++p) {
                    const double m = mask_at(mask, &o, b, t, p);
                    zc res = m * w[p];
                    if (ys) res -= (double)ys[2 * p] + I * (double)ys[2 * p + 1];
                    w[p] = m * res;
                }
                /* 4 (per coil) */
                if (r == ORACLE_OK) r = fft_centered_volume(w, o.n, o.rank, +1);
                for (int64_t p = 0; p < o.V; ++p) {
                    const zc sv = (double)ss[2 * p] + I * (double)ss[2 * p + 1];
                    w[p] = conj(sv) * w[p];
                }
                if (r != ORACLE_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
                    rc = r;
                }
            }
            /* 4 (coil sum, fixed order) and 5 */
            zc* dst = out + (b * o.T + t) * o.V;
            for (int64_t p = 0; p < o.V; ++p) {
                zc a = 0.0;
                for (int64_t c = 0; c < o.C; ++c) a += contrib[c * o.V + p];
                const zc xv = (double)xs[2 * p] + I * (double)xs[2 * p + 1];
                dst[p] = xv - eta * a;
            }
        }
    free(contrib);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * MoDL data-consistency step (the model inversion of Eq. 7, second line):
 *
 *      x = (A^H A + mu I)^{-1} (A^H y + mu z)
 *
 * solved, as the paper states, with the conjugate gradient method and a fixed number of steps
 * (10 in its experiments).  The paper prints no CG listing; this is the textbook method of
 * Hestenes and Stiefel for the Hermitian positive definite system H x = b, H = A^H A + mu I,
 * with the choices the paper leaves open fixed as follows: start at x_0 = 0 (so r_0 = p_0 = b),
 * no preconditioner, exactly n_iter steps, stop early only when the residual is exactly zero,
 * one system per batch example (its frames solved jointly).
 *
 *      alpha_k = <r_k, r_k> / <p_k, H p_k>        x_{k+1} = x_k + alpha_k p_k
 *      r_{k+1} = r_k - alpha_k H p_k              beta_k  = <r_{k+1}, r_{k+1}> / <r_k, r_k>
 *      p_{k+1} = r_{k+1} + beta_k p_k
 * ------------------------------------------------------------------------------------------ */

/* out = A^H A p for a double-precision image p (B,T,V): S_c .* p, F, M .* M, F^H, conj(S_c), coil sum */
static int normal_op(const zc* p, const float* sens, const float* mask, const odims* o, zc* kwork,
                     zc* out, int nthreads)
{
    int rc = ORACLE_OK;
    const int64_t units = o->B * o->C * o->T;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < units; ++u) {
        const int64_t t = u % o->T, c = (u / o->T) % o->C, b = u / (o->T * o->C);
        const zc* ps = p + (b * o->T + t) * o->V;
        const float* ss = sens_ptr(sens, o, b, c, t);
        zc* ku = kwork + u * o->V;
        for (int64_t q = 0; q < o->V; ++q) ku[q] = ((double)ss[2 * q] + I * (double)ss[2 * q + 1]) * ps[q];
        int r = fft_centered_volume(ku, o->n, o->rank, -1);
        for (int64_t q = 0; q < o->V; ++q) {
            const double m = mask_at(mask, o, b, t, q);
            ku[q] = m * (m * ku[q]);
        }
        if (r == ORACLE_OK) r = fft_centered_volume(ku, o->n, o->rank, +1);
        for (int64_t q = 0; q < o->V; ++q) ku[q] = conj((double)ss[2 * q] + I * (double)ss[2 * q + 1]) * ku[q];
        if (r != ORACLE_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc = r;
        }
    }
    for (int64_t b = 0; b < o->B; ++b)
        for (int64_t t = 0; t < o->T; ++t) {
            zc* dst = out + (b * o->T + t) * o->V;
            for (int64_t q = 0; q < o->V; ++q) dst[q] = 0.0;
            for (int64_t c = 0; c < o->C; ++c) {
                const zc* src = kwork + ((b * o->C + c) * o->T + t) * o->V;
                for (int64_t q = 0; q < o->V; ++q) dst[q] += src[q];
            }
        }
    return rc;
}

/* n_iter CG steps on (A^H A + mu I) x = b from x = 0.  b is overwritten (it becomes the residual).
 * Every batch example is its own system (A is block diagonal over the batch): the inner products,
 * alpha and beta are taken per example, over its frames and voxels, so a result does not depend
 * on what else is in the batch.  An example whose residual is exactly zero is left as it is. */
static int cg_solve(zc* b, const float* sens, const float* mask, const odims* o, double mu, int n_iter,
                    zc* x, int nthreads)
{
    const int64_t ne = o->T * o->V;              /* elements of one example */
    const int64_t n = o->B * ne;
    zc* p = (zc*)malloc(sizeof(zc) * (size_t)n);
    zc* Hp = (zc*)malloc(sizeof(zc) * (size_t)n);
    zc* kwork = (zc*)malloc(sizeof(zc) * (size_t)(o->B * o->C * o->T * o->V));
    double* rr = (double*)malloc(sizeof(double) * (size_t)o->B);
    if (!p || !Hp || !kwork || !rr) { free(p); free(Hp); free(kwork); free(rr); return ORACLE_ERR_MEM; }
    int rc = ORACLE_OK;
    zc* r = b;
    for (int64_t e = 0; e < o->B; ++e) {
        rr[e] = 0.0;
        for (int64_t i = e * ne; i < (e + 1) * ne; ++i) {
            x[i] = 0.0; p[i] = r[i];
            rr[e] += creal(r[i]) * creal(r[i]) + cimag(r[i]) * cimag(r[i]);
        }
    }
    for (int k = 0; k < n_iter && rc == ORACLE_OK; ++k) {
        rc = normal_op(p, sens, mask, o, kwork, Hp, nthreads);
        for (int64_t e = 0; e < o->B; ++e) {
            if (!(rr[e] > 0.0)) continue;
            double pHp = 0.0;
            for (int64_t i = e * ne; i < (e + 1) * ne; ++i) {
                Hp[i] += mu * p[i];
                pHp += creal(conj(p[i]) * Hp[i]);
            }
            const double alpha = rr[e] / pHp;
            double rr_new = 0.0;
            for (int64_t i = e * ne; i < (e + 1) * ne; ++i) {
                x[i] += alpha * p[i];
                r[i] -= alpha * Hp[i];
                rr_new += creal(r[i]) * creal(r[i]) + cimag(r[i]) * cimag(r[i]);
            }
            const double beta = rr_new / rr[e];
            for (int64_t i = e * ne; i < (e + 1) * ne; ++i) p[i] = r[i] + beta * p[i];
            rr[e] = rr_new;
        }
    }
    free(p); free(Hp); free(kwork); free(rr);
    return rc;
}

/* x = (A^H A + mu I)^{-1} (A^H y + mu z) by n_iter CG steps (Eq. 7).  z: image (B,T,V), y: k-space. */
int oracle_modl_cg(const float* z, const float* y, const float* sens, const float* mask, double mu, int n_iter,
                   const int64_t* dims, zc* out, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK || !z || !y || !sens || !mask || !out || n_iter < 0) return ORACLE_ERR_ARG;
    const int64_t n = o.B * o.T * o.V, nk = o.B * o.C * o.T * o.V;
    zc* b = (zc*)malloc(sizeof(zc) * (size_t)n);
    zc* k = (zc*)malloc(sizeof(zc) * (size_t)nk);
    if (!b || !k) { free(b); free(k); return ORACLE_ERR_MEM; }
    for (int64_t i = 0; i < nk; ++i) k[i] = (double)y[2 * i] + I * (double)y[2 * i + 1];
    int rc = oracle_apply_AH(k, sens, mask, dims, b, nthreads);          /* b = A^H y */
    free(k);
    for (int64_t i = 0; i < n; ++i) b[i] += mu * ((double)z[2 * i] + I * (double)z[2 * i + 1]);
    if (rc == ORACLE_OK) rc = cg_solve(b, sens, mask, &o, mu, n_iter, out, nthreads);
    free(b);
    return rc;
}

/* Vector-Jacobian product of the step with respect to z, the CG solve taken as the exact inverse
 * (x = H^{-1}(A^H y + mu z), H Hermitian  =>  grad_z = mu H^{-1} g), evaluated by the same number
 * of CG steps:  n_iter steps on H u = mu g  from u = 0. */
int oracle_modl_cg_vjp(const float* g, const float* sens, const float* mask, double mu, int n_iter,
                       const int64_t* dims, zc* out, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK || !g || !sens || !mask || !out || n_iter < 0) return ORACLE_ERR_ARG;
    const int64_t n = o.B * o.T * o.V;
    zc* b = (zc*)malloc(sizeof(zc) * (size_t)n);
    if (!b) return ORACLE_ERR_MEM;
    for (int64_t i = 0; i < n; ++i) b[i] = mu * ((double)g[2 * i] + I * (double)g[2 * i + 1]);
    const int rc = cg_solve(b, sens, mask, &o, mu, n_iter, out, nthreads);
    free(b);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Eq. 3 in its normal-equations form.  A^H (A x - y) = A^H A x - A^H y, so with the zero-filled
 * image  aty = A^H y  given (it does not change over the unrolled iterations of one example)
 *
 *      out = x - eta * (A^H A x - aty).
 *
 * aty: (B, T, n0, n1, n2) single-precision complex, as the GPU call receives it.  Steps: the
 * vector-Jacobian form of oracle_dc gives x - eta A^H A x; eta * aty is added to it.
 * Pins (tests/test_oracle_aty.py): dense-matrix brute force, equality with oracle_dc for
 * aty = A^H y, aty = 0 gives the vector-Jacobian product, exact linearity in aty.
 * ------------------------------------------------------------------------------------------ */
int oracle_dc_aty(const float* x, const float* aty, const float* sens, const float* mask, double eta,
                  const int64_t* dims, zc* out, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK) return ORACLE_ERR_ARG;
    if (!x || !aty || !sens || !mask || !out) return ORACLE_ERR_ARG;
    const int rc = oracle_dc(x, NULL, sens, mask, eta, dims, out, nthreads);
    if (rc != ORACLE_OK) return rc;
    const int64_t total = o.B * o.T * o.V;
    for (int64_t p = 0; p < total; ++p)
        out[p] += eta * ((double)aty[2 * p] + I * (double)aty[2 * p + 1]);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Gradients of the data-consistency step (Eq. 3) with respect to its two other inputs, for a
 * cotangent g of the output (conjugate-Wirtinger convention, as for the vector-Jacobian product
 * with respect to x).  out = x - eta A^H (A x - y) is linear in eta and affine in y, so both are
 * exact:
 *     d out / d eta = -A^H (A x - y)     =>   grad_eta[b] = -Re < g_b , A^H (A x - y)_b >
 *     d out / d y   = +eta A^H           =>   grad_y      = eta A g = eta Omega F S g
 * < u, v > = sum conj(u) v over the frames and voxels of batch example b.  One value per example:
 * a step size shared by the batch takes their sum.
 * ------------------------------------------------------------------------------------------ */
int oracle_dc_grad_eta(const float* g, const float* x, const float* y, const float* sens, const float* mask,
                       const int64_t* dims, double* grad_eta, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK || !g || !x || !y || !sens || !mask || !grad_eta) return ORACLE_ERR_ARG;
    const int64_t n = o.B * o.T * o.V, nk = o.B * o.C * o.T * o.V;
    zc* k = (zc*)malloc(sizeof(zc) * (size_t)nk);
    zc* a = (zc*)malloc(sizeof(zc) * (size_t)n);
    if (!k || !a) { free(k); free(a); return ORACLE_ERR_MEM; }
    int rc = oracle_apply_A(x, sens, mask, dims, k, nthreads);                  /* k = A x */
    for (int64_t i = 0; i < nk; ++i) k[i] -= (double)y[2 * i] + I * (double)y[2 * i + 1];   /* A x - y */
    if (rc == ORACLE_OK) rc = oracle_apply_AH(k, sens, mask, dims, a, nthreads);   /* a = A^H (A x - y) */
    const int64_t ne = o.T * o.V;
    for (int64_t b = 0; b < o.B; ++b) {
        double acc = 0.0;
        for (int64_t i = b * ne; i < (b + 1) * ne; ++i) {
            const zc gv = (double)g[2 * i] + I * (double)g[2 * i + 1];
            acc += creal(conj(gv) * a[i]);
        }
        grad_eta[b] = -acc;
    }
    free(k); free(a);
    return rc;
}

int oracle_dc_grad_y(const float* g, const float* sens, const float* mask, double eta, const int64_t* dims,
                     zc* grad_y, int nthreads)
{
    odims o;
    if (parse_dims(dims, &o) != ORACLE_OK || !g || !sens || !mask || !grad_y) return ORACLE_ERR_ARG;
    const int rc = oracle_apply_A(g, sens, mask, dims, grad_y, nthreads);       /* A g */
    const int64_t nk = o.B * o.C * o.T * o.V;
    for (int64_t i = 0; i < nk; ++i) grad_y[i] *= eta;
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Bridge to the learned prior.  The paper's networks take a complex image as two real channels
 * (real part, imaginary part) and are trained with an l1 loss on complex images (Implementation /
 * Training).  Readings: the channel axis sits right after the batch axis,
 *      complex (B, T, n0, n1, n2)   <->   real (B, 2, T, n0, n1, n2),  channel 0 = Re, 1 = Im;
 * the loss is the mean modulus of the difference over all B T V complex elements,
 *      L = (1 / N) sum_i | x_i - r_i | ;
 * its gradient in the conjugate-Wirtinger convention (the one a real loss back-propagates through
 * complex tensors, 2 dL/d conj(x)) is (x_i - r_i) / |x_i - r_i| / N, and zero where x_i = r_i.
 * ------------------------------------------------------------------------------------------ */
void oracle_complex_to_channels(const float* x, int64_t B, int64_t inner, float* out)
{
    for (int64_t b = 0; b < B; ++b)
        for (int64_t i = 0; i < inner; ++i) {
            out[(b * 2 + 0) * inner + i] = x[2 * (b * inner + i)];
            out[(b * 2 + 1) * inner + i] = x[2 * (b * inner + i) + 1];
        }
}

void oracle_channels_to_complex(const float* ch, int64_t B, int64_t inner, float* out)
{
    for (int64_t b = 0; b < B; ++b)
        for (int64_t i = 0; i < inner; ++i) {
            out[2 * (b * inner + i)] = ch[(b * 2 + 0) * inner + i];
            out[2 * (b * inner + i) + 1] = ch[(b * 2 + 1) * inner + i];
        }
}

/* mean | x - r | over n complex elements; grad (optional, n complex doubles) as stated above */
double oracle_l1_loss(const float* x, const float* r, int64_t n, zc* grad)
{
    double sum = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const zc d = ((double)x[2 * i] - (double)r[2 * i]) + I * ((double)x[2 * i + 1] - (double)r[2 * i + 1]);
        const double m = cabs(d);
        sum += m;
        if (grad) grad[i] = (m > 0.0) ? d / m / (double)n : 0.0;
    }
    return sum / (double)n;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
