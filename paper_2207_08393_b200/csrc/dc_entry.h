// Entry points of the data-consistency path that other translation units of the library use.
#pragma once
#include <cuda_runtime.h>
#include "../../include/gleam.h"

namespace gleam {

// RUN_PREPARE: only what depends on y and the mask alone (rank map, z table) is computed and left in
// the workspace; RUN_APPLY: the step with those tables taken from the workspace as they are.
enum { RUN_ALL = 0, RUN_PREPARE = 1, RUN_APPLY = 2 };

// out = x - eta A^H (A x - y)   (y == nullptr: out = x - eta A^H A x).  Validates its arguments,
// enqueues on d->stream, returns GLEAM_OK or a GLEAM_ERR_* code.  check_only: the argument checks
// alone (callers that must enqueue something of their own before the step run them first).
int run(const void* x, const void* y, const void* sens, const float* mask, float eta, void* out,
        const gleam_dims* d, int mode = RUN_ALL, double* dot_rows = nullptr, bool check_only = false,
        int layout = 0,      // layout: GLEAM_X_CHANNELS | GLEAM_OUT_CHANNELS (two-real-channel image arrays)
        const void* aty = nullptr);   // with y == nullptr: out = x - eta (A^H A x - aty), aty = A^H y as an image

// dot_rows (device, one double per image row, B*T*n1): the one-pass 2-D kernel also stores
// Re<x_row, out_row> of every row it writes, so that a caller's inner product <x, out> needs no
// pass of its own.  Only where this returns true (2-D, readout-invariant mask, warp-resident row plan).
bool dot_rows_supported(const gleam_dims* d);

// GLEAM_OK for a device (or managed) pointer, GLEAM_ERR_NOT_DEVICE_POINTER otherwise
int check_device_ptr(const void* p);

// counts a launch of kernel class cls and, while per-kernel timing is on, records its event
cudaError_t prof_mark(int cls, cudaStream_t s);

}  // namespace gleam
