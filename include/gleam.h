/*
 * gleam.h — C ABI of the B200 (sm_100a) multi-coil SENSE data-consistency library.
 *
 * The library computes the data-consistency step of the unrolled proximal-gradient network of
 * GLEAM (arXiv 2207.08393) and its vector-Jacobian product:
 *
 *     sensing model (Eq. 1)            y = Omega F S x + eps
 *     forward operator (after Eq. 2)   A = Omega F S,  A^H its Hermitian transpose
 *     data consistency (Eq. 3)         DC(x) = x - 2t A^H (A x - y)            eta := 2t
 *     Jacobian of Eq. 3                J = I - eta A^H A   (Hermitian for real eta)
 *
 * S multiplies the image by each coil's sensitivity map, F is the centred orthonormal DFT over the
 * trailing fft_rank spatial axes (centre index floor(N/2) in both domains, kernel
 * exp(-2 pi i (k-o)(n-o)/N) / sqrt(N)), Omega multiplies k-space by a real sampling weight
 * (normally 0/1).  Omega is applied once in A and once more in A^H, as the definition says:
 * r_c = M .* (M .* F(S_c .* x) - y_c).
 *
 * Data layout: every array is contiguous, row-major, last index fastest.  complex64 means
 * interleaved {float re, float im}.
 *     x, out, grad_out, grad_in : (B, T, n0, n1, n2)           complex64
 *     y                         : (B, C, T, n0, n1, n2)        complex64
 *     sens                      : (B, C, n0, n1, n2) or (B, C, T, n0, n1, n2)   complex64
 *     mask                      : see mask_kind                 float32
 * B batch, C coils, T frames (never transformed), n0 = 1 when fft_rank == 2.
 *
 * Ownership: all data pointers are DEVICE pointers owned by the caller.  The library neither
 * allocates nor frees device memory and keeps no pointer after the call returns.  Work is
 * enqueued on dims->stream and the call returns without synchronising; the buffers (including the
 * workspace) must stay valid and untouched until that work has completed.
 *
 * Errors: every function returns GLEAM_OK (0) or a negative GLEAM_ERR_* code.  Argument checks
 * run on the host before anything is enqueued; a call that returns an argument error has launched
 * nothing.  GLEAM_ERR_CUDA reports a failed launch; kernels enqueued before it may still run.
 * Unsupported transform lengths are reported (GLEAM_ERR_UNSUPPORTED_SIZE), never emulated on the
 * CPU.  Results are deterministic: the same inputs give bit-identical outputs on every call.
 */
#ifndef GLEAM_H_
#define GLEAM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define GLEAM_API __attribute__((visibility("default")))
#else
#define GLEAM_API
#endif

#define GLEAM_VERSION 1
#define GLEAM_DIMS_VERSION 1

enum {
    GLEAM_OK = 0,
    GLEAM_ERR_NULL_POINTER = -1,
    GLEAM_ERR_BAD_DIMS = -2,
    GLEAM_ERR_UNSUPPORTED_SIZE = -3,
    GLEAM_ERR_NOT_DEVICE_POINTER = -4,
    GLEAM_ERR_WORKSPACE_TOO_SMALL = -5,
    GLEAM_ERR_ALIAS = -6,
    GLEAM_ERR_CUDA = -7,
    GLEAM_ERR_UNIMPLEMENTED = -8,
    GLEAM_ERR_TIMEOUT = -9
};

enum {
    GLEAM_MASK_FULL = 0,             /* mask is (B, T, n0, n1, n2) */
    GLEAM_MASK_READOUT_INVARIANT = 1 /* mask does not depend on the readout index:
                                        fft_rank 2 -> (B, T, n2)      (readout axis n1)
                                        fft_rank 3 -> (B, T, n1, n2)  (readout axis n0) */
};

typedef struct {
    int32_t struct_version;  /* GLEAM_DIMS_VERSION */
    int32_t batch;           /* B >= 1 */
    int32_t coils;           /* C >= 1 */
    int32_t frames;          /* T >= 1; the frame axis is not transformed */
    int32_t fft_rank;        /* 2 or 3 */
    int32_t n[3];            /* n0, n1, n2 (slowest to fastest); n0 = 1 when fft_rank == 2 */
    int32_t sens_has_frames; /* 0: sens is (B,C,n0,n1,n2); 1: (B,C,T,n0,n1,n2) */
    int32_t mask_kind;       /* GLEAM_MASK_* ; the mask is broadcast over coils */
    void* stream;            /* cudaStream_t; NULL = the legacy default stream */
    void* workspace;         /* device scratch of at least gleam_dc_workspace_size() bytes,
                                256-byte aligned; its contents are undefined afterwards */
    uint64_t workspace_bytes;
} gleam_dims;

/*
 * Data-consistency step, Eq. 3:   out = x - eta * A^H (A x - y).
 *   x, y, sens, mask, out : device pointers, layouts above.  out may be exactly x (in place);
 *   any other overlap between an output or the workspace and another argument is
 *   GLEAM_ERR_ALIAS.  y may hold anything where the mask is zero: those samples are not read.
 *   eta : real step size (2t in the paper's notation).
 */
GLEAM_API int gleam_dc_forward(const void* x, const void* y, const void* sens, const float* mask, float eta,
                     void* out, const gleam_dims* dims);

/*
 * Vector-Jacobian product of Eq. 3 with respect to x:   grad_in = grad_out - eta * A^H A grad_out
 * (J^H g with J = I - eta A^H A; the conjugate-Wirtinger convention for complex tensors).
 * grad_in may be exactly grad_out.
 */
GLEAM_API int gleam_dc_vjp(const void* grad_out, const void* sens, const float* mask, float eta,
                 void* grad_in, const gleam_dims* dims);

/*
 * Scratch bytes that gleam_dc_forward / gleam_dc_vjp need for these dims (the larger of the two).
 * Reads only the shape fields of dims; stream and workspace are ignored.
 */
GLEAM_API int gleam_dc_workspace_size(const gleam_dims* dims, uint64_t* bytes);

/*
 * Device-side status of the work enqueued so far with these dims and this workspace (the paper has
 * no counterpart).  The separable 3-D path (fft_rank 3, readout-invariant mask, n2 = 256 and n1 a
 * compiled multiple of 16) runs Eq. 3 as one persistent kernel whose blocks hand slabs of the coil
 * workspace to one another through L2; every wait of one block for another is bounded (two seconds).
 * A wait that runs out makes the kernel stop early and leaves an error word in the workspace.  This
 * call synchronises dims->stream, reads the word and returns GLEAM_ERR_TIMEOUT if it is set (the
 * output of that call is then undefined), GLEAM_OK otherwise.  For every other problem class it
 * only synchronises and returns GLEAM_OK: no other kernel waits on another block.
 */
GLEAM_API int gleam_dc_check_status(const gleam_dims* dims);

/*
 * Which kernels the separable 3-D path uses for phase-encode extents (n1, n2): the number of rows RY a block
 * of the row-tile kernels holds (n1 = RY * BY; every pass over the workspace contiguous), or 0 when the pair
 * has no row-tile kernels and the general strided middle pass is used.  Informational.
 */
GLEAM_API int32_t gleam_dc_rowtile_split(int32_t n1, int32_t n2);

/*
 * Selects (on != 0) or deselects the persistent kernel for the problem class described above; the default
 * is off unless the environment holds GLEAM_FUSED=1, because the three whole-volume passes measure faster
 * on one B200.  Process-wide; call it before gleam_dc_workspace_size (the scratch layout depends on it).
 */
GLEAM_API void gleam_dc_set_fused(int32_t on);

/*
 * Measurement aid: how long the blocks of the last persistent-kernel call with these dims and workspace
 * waited, summed over all blocks.  ns_and_counts receives n_kinds (<= 5) pairs {nanoseconds, waits that
 * had to spin}: 0 a ring slot to become free, 1 the first pass of a slab to complete, 2 the middle pass
 * to complete (all three: one block waiting for others), 3 and 4 a staged tile (sensitivities / workspace)
 * that had not landed when a compute group needed it.  Synchronises dims->stream.
 */
GLEAM_API int gleam_dc_fused_wait_stats(const gleam_dims* dims, uint64_t* ns_and_counts, int32_t n_kinds);

/*
 * Test aid for the bounded waits above: the item with this number (>= 0) of the persistent kernel is
 * drawn but neither run nor counted as done, so that the blocks depending on it run into their wait
 * limit; wait_limit_ns shortens the limit (0 = the default).  (-1, 0) restores normal operation.
 * Process-wide; not for production use.
 */
GLEAM_API void gleam_dc_debug_fused(int32_t withhold_item, uint64_t wait_limit_ns);

/*
 * GLEAM_OK if a transform of this length is supported along an axis (even lengths whose plan is
 * compiled in), GLEAM_ERR_UNSUPPORTED_SIZE otherwise.
 */
GLEAM_API int gleam_dc_length_supported(int32_t n);

/*
 * Host-buffer variants of the two calls above (no counterpart in the paper: a convenience for
 * callers whose data lives in host memory).  x, y, sens, mask, out are HOST pointers with the same
 * layouts; pinned memory makes the copies asynchronous.  `arena` is a DEVICE buffer of at least
 * gleam_dc_host_arena_size() bytes, 256-byte aligned, that holds the staged inputs, the output and
 * the workspace; dims->workspace is ignored.  The calls enqueue, on dims->stream, the
 * host-to-device copies, the kernels and the device-to-host copy of the result, and return
 * without synchronising: out is valid once the stream has drained.
 */
GLEAM_API int gleam_dc_forward_host(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                    void* out, const gleam_dims* dims, void* arena, uint64_t arena_bytes);
GLEAM_API int gleam_dc_vjp_host(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_in,
                                const gleam_dims* dims, void* arena, uint64_t arena_bytes);
GLEAM_API int gleam_dc_host_arena_size(const gleam_dims* dims, uint64_t* bytes);

/*
 * gleam_dc_forward_static: gleam_dc_forward for callers that must not allocate device memory.
 * (The paper has no counterpart; this is a deployment convenience.)  Some users of this library
 * run where cudaMalloc is off the table: a reconstruction service whose device memory was handed
 * out in full to a framework's caching allocator at start-up, a plug-in that may touch only the
 * buffers its host application passes in, a real-time loop in which an allocation's implicit
 * device synchronisation is unacceptable.  For them the scratch that gleam_dc_forward takes from
 * dims->workspace lives inside the library instead, in one fixed device array of
 * gleam_dc_static_scratch_bytes() bytes (64 MiB) that every GPU loading the library keeps until
 * the process exits.  dims->workspace and dims->workspace_bytes are ignored; inputs and the
 * output are still the caller's device buffers, with the layouts and rules of gleam_dc_forward.
 *   - Problems whose scratch need (gleam_dc_workspace_size) exceeds the array return
 *     GLEAM_ERR_WORKSPACE_TOO_SMALL and launch nothing.
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current); make that first call before any stream capture begins.  With CUDA's lazy module
 *     loading the array itself comes into being when the library's device code is first loaded on a
 *     device, which may be that first call (or any earlier call of this library there): that one
 *     call can then take device memory and synchronise implicitly, and fails with GLEAM_ERR_CUDA if
 *     64 MiB are no longer free.  Make it at start-up, before the device's memory is handed out;
 *     every later call leaves the amount of free device memory unchanged.
 *   - All calls share the one array, which keeps whatever the previous call left in it; the
 *     kernels write every scratch element before reading it, so no clearing is needed.  Two calls
 *     whose GPU work overlaps (different streams, or different host threads on one device) race on
 *     the array and give undefined results: order them on one stream or with events.
 */
GLEAM_API int gleam_dc_forward_static(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                      void* out, const gleam_dims* dims);
GLEAM_API uint64_t gleam_dc_static_scratch_bytes(void);

/* ---- unrolled iterations with the same measurements -------------------------------------------
 * Every unrolled iteration (and every greedy module of Alg. 1) applies Eq. 3 with the same y and
 * mask.  For a readout-invariant mask, what the step needs from y does not depend on x: the table
 * z = M R^H y at the sampled phase-encode positions (R = transform along the readout axis) and the
 * rank map of those positions.  gleam_dc_prepare computes both into dims->workspace;
 * gleam_dc_forward_prepared then gives exactly the result of gleam_dc_forward (bit for bit) without
 * recomputing them.  Between the two, the caller keeps that workspace untouched: no other call of
 * this library may be given it (a gleam_dc_vjp in between needs a workspace of its own), and the
 * mask and dims must be the same.  With GLEAM_MASK_FULL there is nothing to prepare: _prepare does
 * nothing and _forward_prepared is gleam_dc_forward.  y is passed to both (it is read by
 * _forward_prepared only for a full mask).  Errors as for gleam_dc_forward.
 */
GLEAM_API int gleam_dc_prepare(const void* y, const float* mask, const gleam_dims* dims);
GLEAM_API int gleam_dc_forward_prepared(const void* x, const void* y, const void* sens, const float* mask,
                                        float eta, void* out, const gleam_dims* dims);

/* ---- the step in its normal-equations form ----------------------------------------------------
 * A^H (A x - y) = A^H A x - A^H y, so Eq. 3 is also
 *
 *      out = x - eta * (A^H A x - aty),        aty = A^H y   (gleam_dc_adjoint),
 *
 * and the zero-filled image A^H y of an example is the same for all unrolled iterations and all
 * greedy modules of Alg. 1 (it is the usual starting image x^0 as well).  With it given, a step
 * costs what gleam_dc_vjp costs: no pass over y, no table of y, no per-sample look-up.
 *   aty : device, complex64, (B, T, n0, n1, n2), 16-byte aligned; may alias x, must not overlap out
 *         or the workspace.  Any image is accepted (the call evaluates the formula above).
 * Other arguments, workspace (that of gleam_dc_vjp), in-place rule (out == x allowed) and errors
 * as for gleam_dc_forward.  The vector-Jacobian product with respect to x is gleam_dc_vjp; the
 * cotangent of aty is eta * grad_out.  The result equals gleam_dc_forward(x, y, ...) up to
 * single-precision rounding (different order of operations), not bit for bit.
 */
GLEAM_API int gleam_dc_forward_aty(const void* x, const void* aty, const void* sens, const float* mask, float eta,
                                   void* out, const gleam_dims* dims);

/* ---- zero-filled SENSE image -----------------------------------------------------------------
 * out = A^H y = sum_c conj(S_c) F^H (Omega y_c): the image the paper's networks start from (its
 * Experiments section feeds "zero-filled, SENSE-reconstructed" images).  Evaluated as Eq. 3 on a
 * zero image with eta = 1; arguments, workspace and errors as for gleam_dc_forward.
 */
GLEAM_API int gleam_dc_adjoint(const void* y, const void* sens, const float* mask, void* out,
                               const gleam_dims* dims);

/* ---- bridge to the learned prior ---------------------------------------------------------------------
 * The paper's networks take and return complex images as two real channels (real part, imaginary part;
 * Implementation / Training) and are trained with an l1 loss on complex images.  The _layout variants of
 * the two main calls read and / or write the image-side arrays directly in that form,
 *     (B, 2, T, n0, n1, n2) float32, channel 0 = real part, channel 1 = imaginary part,
 * inside the kernels that load x and store out, so no conversion pass is needed on either side of the
 * prior.  layout: GLEAM_X_CHANNELS (x / grad_out is two-channel), GLEAM_OUT_CHANNELS (out / grad_in is);
 * 0 gives gleam_dc_forward / gleam_dc_vjp.  In place (out == x) needs both or neither.  With a layout flag
 * the opt-in persistent kernel is not used.
 *
 * gleam_l1_loss:  loss = mean over all B T n0 n1 n2 complex elements of |x - ref|  (device double), and, if
 * grad is not null, grad = (x - ref) / |x - ref| / N, zero where x = ref: the gradient a real loss sends
 * back through a complex tensor (conjugate-Wirtinger convention), in the layout GLEAM_OUT_CHANNELS selects.
 * ref is complex64 (B, T, n0, n1, n2); x in the layout GLEAM_X_CHANNELS selects.  The mean is accumulated in
 * double precision in a fixed order.  dims->workspace: gleam_l1_loss_workspace_size() bytes.
 */
#define GLEAM_X_CHANNELS 1u
#define GLEAM_OUT_CHANNELS 2u
GLEAM_API int gleam_dc_forward_layout(const void* x, const void* y, const void* sens, const float* mask, float eta,
                                      void* out, const gleam_dims* dims, uint32_t layout);
GLEAM_API int gleam_dc_vjp_layout(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_in,
                                  const gleam_dims* dims, uint32_t layout);
GLEAM_API int gleam_l1_loss(const void* x, const void* ref, double* loss, void* grad, const gleam_dims* dims,
                            uint32_t layout);
GLEAM_API uint64_t gleam_l1_loss_workspace_size(void);

/* ---- gradients of Eq. 3 with respect to the step size and the measurements --------------------------
 * out = x - eta A^H (A x - y) is linear in eta and affine in y.  For a cotangent g = grad_out of the
 * output (conjugate-Wirtinger convention, as for gleam_dc_vjp):
 *     grad_eta[b] = -Re < g_b , A^H (A x - y)_b >        one double per batch example (device, B values);
 *                                                        a step size shared by the batch takes their sum
 *     grad_y      = eta A g = eta Omega F S g             complex64, layout of y; zero where the mask is zero
 * The paper does not say whether the step size 2t of Eq. 3 is trained; these are the exact derivatives
 * for a caller that trains it, or that needs the sensitivity of the step to the measurements.
 * dims->workspace: gleam_dc_grad_workspace_size bytes.  grad_eta evaluates the step once with eta = 1
 * (all kernels of gleam_dc_forward) and reduces in double precision in a fixed order; grad_y runs the
 * forward operator alone.  Argument rules and errors as for gleam_dc_forward; nothing may overlap an
 * output or the workspace.
 */
GLEAM_API int gleam_dc_grad_eta(const void* grad_out, const void* x, const void* y, const void* sens, const float* mask,
                                double* grad_eta, const gleam_dims* dims);
GLEAM_API int gleam_dc_grad_y(const void* grad_out, const void* sens, const float* mask, float eta, void* grad_y,
                              const gleam_dims* dims);
GLEAM_API int gleam_dc_grad_workspace_size(const gleam_dims* dims, uint64_t* bytes);

/* ---- MoDL data-consistency step (Eq. 7, second line) -------------------------------------------
 *
 *     out = (A^H A + mu I)^{-1} (A^H y + mu z)
 *
 * by n_iter conjugate-gradient steps (the paper's experiments use 10), A = Omega F S as above.  The
 * paper prints no CG listing; the choices it leaves open are fixed as: start from zero, no
 * preconditioner, exactly n_iter steps, one system per batch example (inner products over the
 * example's frames and voxels, so a result does not depend on the rest of the batch), an example
 * whose residual is exactly zero is left as it is.
 *
 *   z, out   : device, complex64 (B,T,n0,n1,n2); out == z (exact alias) is allowed
 *   y, sens, mask, dims : as for gleam_dc_forward
 *   mu       : > 0 (GLEAM_ERR_BAD_DIMS otherwise); n_iter in [0, 1000]; n_iter = 0 gives out = 0
 *   dims->workspace: gleam_modl_cg_workspace_size bytes (the data-consistency workspace, three
 *              image-sized vectors and the reduction scratch)
 *
 * gleam_modl_cg_vjp is the vector-Jacobian product with respect to z with the solve taken as the
 * exact inverse (the Jacobian mu (A^H A + mu I)^{-1} is Hermitian):
 *     grad_z = mu (A^H A + mu I)^{-1} grad_out     by n_iter conjugate-gradient steps from zero.
 * Inner products are accumulated in double precision in a fixed order: results are deterministic.
 * Everything is enqueued on dims->stream; no allocation, no synchronisation.
 */
GLEAM_API int gleam_modl_cg_forward(const void* z, const void* y, const void* sens, const float* mask, float mu,
                                    int32_t n_iter, void* out, const gleam_dims* dims);
GLEAM_API int gleam_modl_cg_vjp(const void* grad_out, const void* sens, const float* mask, float mu,
                                int32_t n_iter, void* grad_z, const gleam_dims* dims);
GLEAM_API int gleam_modl_cg_workspace_size(const gleam_dims* dims, uint64_t* bytes);

/*
 * Measurement aids (no counterpart in the paper).
 * gleam_dc_launch_count: kernels this library has launched since it was loaded.
 * gleam_dc_profile_begin / _end: between the two, every kernel launch is bracketed by CUDA events
 * on its stream; _end waits for the last one and returns, per kernel class GLEAM_K_*, the summed
 * device time in milliseconds and the number of launches (arrays of n_classes entries).
 * Profiling creates CUDA events on first use and is meant for benchmarks, not for production.
 */
enum {
    GLEAM_K_PREP_M2 = 0,      /* rank map of the sampled positions (forward call only) */
    GLEAM_K_COL_Z = 1,        /* readout-axis inverse transform of y */
    GLEAM_K_ROW_FUSED = 2,    /* 2-D one-pass kernel */
    GLEAM_K_ROW_FWD = 3,      /* sensitivity multiply + transform of the contiguous axis */
    GLEAM_K_COL_MID_SEP = 4,  /* strided axis forward, mask/residual, inverse (separable path) */
    GLEAM_K_ROW_INV = 5,      /* inverse of the contiguous axis + coil sum + update */
    GLEAM_K_COL_MID_FULL = 6, /* same as 4 for a full mask */
    GLEAM_K_COL_FWD = 7,
    GLEAM_K_COL_INV = 8,
    GLEAM_K_CG_VEC = 9,       /* image-sized vector kernels of the conjugate-gradient solve */
    GLEAM_K_FUSED3D = 10,     /* persistent kernel of the separable 3-D path (all three passes) */
    GLEAM_K_CLASSES = 11
};
GLEAM_API uint64_t gleam_dc_launch_count(void);
/* FP32 FMA throughput of the current device in TFLOP/s (2 flop per FMA), from a kernel of independent FMA
 * chains without memory traffic, best of four timed launches: the measured ALU peak the benchmark reports
 * beside the nominal one.  scratch4: at least 4 device bytes (never written).  Synchronises the stream. */
GLEAM_API int gleam_measure_fp32_peak(void* scratch4, void* stream, double* tflops);
GLEAM_API int gleam_dc_profile_begin(void);
GLEAM_API int gleam_dc_profile_end(float* ms, uint32_t* launches, int32_t n_classes);

/* Static, human-readable text for a status code. */
GLEAM_API const char* gleam_status_string(int status);

/* GLEAM_VERSION of the loaded library. */
GLEAM_API int gleam_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GLEAM_H_ */
