// Internal interface between the two translation units of libcocod.so (not part of the C boundary):
// lets the MLP gradient path apply a local step itself, inside its weight-gradient kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cocod.h"

struct cocod_step_plan {
    const float *x_in;        // where x lives now
    float *x_out;             // where this step must leave x (differs from x_in right after comm_begin)
    float *v;
    __nv_bfloat16 *shadow;    // bf16 copy of x to keep current (may be NULL)
    float lr, mu, wd;
    int K;
    int64_t P;
    cudaStream_t compute;
};

// Describe the local step the engine would run now.  Fails like cocod_local_step would.
int cocod_internal_plan_step(cocod_handle *h, cocod_step_plan *plan);

// Account for a completed local step (buffer flip, step counter).
int cocod_internal_finish_step(cocod_handle *h, int kernels_launched);
