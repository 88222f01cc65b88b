// Dispatch of the depthwise kernels and of the tcgen05 GEMM / implicit-GEMM kernels: each
// function decides whether the shape qualifies and, if so, enqueues the fast kernel.
#include <cstdio>

#include "qasr_host.h"

int qasr_gemm_tc_init(qasr_ctx* ctx);
int qasr_launch_gemm_tc(qasr_ctx* ctx, const QasrConvArgs& a);
int qasr_launch_dw_dp4a(qasr_ctx* ctx, const QasrDwArgs& a);
int qasr_dw_tc_init(qasr_ctx* ctx);
int qasr_launch_dw_tc(qasr_ctx* ctx, const QasrDwArgs& a);
int qasr_conv_tc_init(qasr_ctx* ctx);
int qasr_launch_conv_tc(qasr_ctx* ctx, const QasrConvArgs& a);

static inline bool al16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

int qasr_host_init(qasr_ctx* ctx) {
    if (ctx->cc_major != 10) {   // the tensor-core and TMA kernels are sm_100a code
        ctx->opt_tc = false;
        return QASR_OK;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    ctx->encode_tiled = fn;
    int rc = qasr_gemm_tc_init(ctx);
    if (rc != QASR_OK) return rc;
    rc = qasr_dw_tc_init(ctx);
    if (rc != QASR_OK) return rc;
    return qasr_conv_tc_init(ctx);
}

int qasr_try_dw_fast(qasr_ctx* ctx, const QasrDwArgs& a) {
    if (!ctx->opt_tc) return 0;   // option 0 forces the generic kernels everywhere
    if (ctx->encode_tiled) {      // sm_100: banded GEMM on the tensor cores
        int used = qasr_launch_dw_tc(ctx, a);
        if (used != 0) return used;
    }
    return qasr_launch_dw_dp4a(ctx, a);
}

bool qasr_conv_shape_fits_gemm(int C_in, int K, int stride, int dilation, int T_out) {
    return K == 1 && stride == 1 && dilation == 1 && C_in % 64 == 0 && C_in <= 1024 && T_out % 16 == 0 && T_out >= 16;
}

int qasr_try_conv_tc(qasr_ctx* ctx, const QasrConvArgs& a) {
    if (!ctx->opt_tc || !ctx->encode_tiled) return 0;
    if (a.T_out % 16 != 0 || a.T_out < 16) return 0;
    if (!al16(a.x) || (a.y && !al16(a.y)) || (a.y_int32 && !al16(a.y_int32))) return 0;
    for (int j = 1; j < a.terms.n; ++j)
        if (!al16(a.terms.ptr[j])) return 0;
    if (qasr_conv_shape_fits_gemm(a.C_in, a.K, a.stride, a.dilation, a.T_out) && al16(a.w)) {
        int rc = qasr_launch_gemm_tc(ctx, a);   // pointwise: activations stay in their own layout
        return rc == QASR_OK ? 1 : rc;
    }
    return qasr_launch_conv_tc(ctx, a);         // K taps / stride / odd channel counts: implicit GEMM, needs scratch
}
