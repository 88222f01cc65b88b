// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/qasr.h"

// Device status word bits (sticky, OR-ed by kernels, read by qasr_poll_status).
#define QASR_STATUS_RANGE 1u    // a shift outside [1,62] or a negative multiplier was seen
#define QASR_STATUS_TIMEOUT 2u  // a bounded device-side wait expired

// Residual terms of a fused epilogue / a standalone add: per-tensor constants by value.
struct QasrTerms {
    int32_t n;                          // 0 = no residual stage
    const int8_t* ptr[QASR_MAX_TERMS];  // ptr[0] unused in a conv epilogue (main branch)
    int32_t mult[QASR_MAX_TERMS];
    int32_t shift[QASR_MAX_TERMS];
};

// Constant arrays (weights, bias, multipliers, shifts) of the kernel that follows in the stream: the running
// kernel asks the L2 to fetch them, so that the next one does not start on DRAM latency.
#define QASR_PREFETCH_RANGES 4
struct QasrPrefetch {
    const void* ptr[QASR_PREFETCH_RANGES];
    uint32_t bytes[QASR_PREFETCH_RANGES];
};

// Arguments of one convolution launch (pointwise or dense), after validation.
struct QasrConvArgs {
    const int8_t* x;
    const int8_t* w;
    const int32_t* bias;
    const int32_t* mult;
    const uint8_t* shift;
    int8_t* y;
    int32_t* y_int32;
    int B, C_in, C_out, T, T_out, K, stride, dilation, relu;
    QasrTerms terms;
    void* scratch;            // optional device scratch for the tensor-core path of a K-tap convolution
    size_t scratch_bytes;
    void* wt;                 // optional separate home of the regrouped weights (else they follow the input copy in scratch)
    int wt_ready;             // wt already holds this layer's regrouped weights: skip the regrouping kernel
    int8_t* yt;               // optional second home of the output, frame-major [B][T_out][C_out]: what a K-tap
                              // convolution that reads this tensor next (stride 1) wants as its input copy
    int xt_ready;             // scratch already holds this layer's frame-major input copy: skip the transpose
};

struct QasrDwArgs {
    const int8_t* x;
    const int8_t* w;
    const int32_t* mult;
    const uint8_t* shift;
    int8_t* y;
    int B, C, T, T_out, K, stride, dilation;
};

// Generic kernels: any shape, any alignment.
cudaError_t qasr_launch_dw_generic(const QasrDwArgs& a, unsigned* status, cudaStream_t st);
cudaError_t qasr_launch_conv_generic(const QasrConvArgs& a, unsigned* status, cudaStream_t st);
cudaError_t qasr_launch_residual_add(const QasrTerms& t, size_t n, int relu, int8_t* y,
                                     unsigned* status, cudaStream_t st);
cudaError_t qasr_launch_glu(const int8_t* x, int B, int C, int T, int q_c, const int32_t* mult,
                            const uint8_t* shift, int8_t* y, unsigned* status, cudaStream_t st, int early_launch = 0);
cudaError_t qasr_launch_dequant(const int32_t* acc, int B, int C, int T, const float* scale,
                                float* out, cudaStream_t st);
