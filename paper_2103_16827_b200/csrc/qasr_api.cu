// C-ABI entry points: context, argument validation, dispatch, layer-table interpreter.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "qasr_internal.h"
#include "qasr_host.h"

// ------------------------------------------------------------------------------------------
// context
// ------------------------------------------------------------------------------------------
static void set_err(qasr_ctx* ctx, const char* fmt, ...) {
    if (!ctx) return;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
}

#define QASR_FAIL(ctx, code, ...)      \
    do {                               \
        set_err((ctx), __VA_ARGS__);   \
        return (code);                 \
    } while (0)

#define QASR_CUDA(ctx, expr)                                                              \
    do {                                                                                  \
        cudaError_t e_ = (expr);                                                          \
        if (e_ != cudaSuccess) {                                                          \
            set_err((ctx), "%s failed: %s", #expr, cudaGetErrorString(e_));               \
            return QASR_ERR_CUDA;                                                         \
        }                                                                                 \
    } while (0)

extern "C" const char* qasr_strerror(int code) {
    switch (code) {
        case QASR_OK: return "ok";
        case QASR_ERR_NULL: return "a required pointer is NULL";
        case QASR_ERR_SHAPE: return "invalid shape or convolution parameter";
        case QASR_ERR_ALIGN: return "pointer alignment";
        case QASR_ERR_RANGE: return "requantisation constant out of range";
        case QASR_ERR_OVERFLOW_RISK: return "int32 accumulator overflow cannot be excluded";
        case QASR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case QASR_ERR_CUDA: return "CUDA call failed";
        case QASR_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
        case QASR_ERR_TABLE: return "inconsistent layer table";
        case QASR_ERR_ALIAS: return "output aliases an input";
        case QASR_ERR_TOO_LARGE: return "operation exceeds the static scratch of the allocation-free entry point";
        default: return "unknown error code";
    }
}

extern "C" int qasr_create(qasr_ctx** out, int device, void* cuda_stream) {
    if (!out) return QASR_ERR_NULL;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return QASR_ERR_CUDA;
    qasr_ctx* ctx = new (std::nothrow) qasr_ctx();
    if (!ctx) return QASR_ERR_CUDA;
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    if (cudaSetDevice(device) != cudaSuccess || cudaMalloc(&ctx->d_status, 256) != cudaSuccess ||
        cudaMemset(ctx->d_status, 0, 256) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return QASR_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) {
        ctx->sm_count = prop.multiProcessorCount;
        ctx->cc_major = prop.major;
    }
    int rc = qasr_host_init(ctx);
    if (rc != QASR_OK) {
        cudaFree(ctx->d_status);
        delete ctx;
        return rc;
    }
    *out = ctx;
    return QASR_OK;
}

extern "C" int qasr_destroy(qasr_ctx* ctx) {
    if (!ctx) return QASR_ERR_NULL;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    qasr_plan_cache_clear(ctx);
    for (QasrProfRec& r : ctx->prof) {
        cudaEventDestroy(r.e0);
        cudaEventDestroy(r.e1);
    }
    if (ctx->capture_stream) cudaStreamDestroy(ctx->capture_stream);
    if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_side) cudaEventDestroy(ctx->ev_side);
    if (ctx->copy_in) cudaStreamSynchronize(ctx->copy_in);
    if (ctx->copy_out) cudaStreamSynchronize(ctx->copy_out);
    for (int s = 0; s < 2; ++s) {
        if (ctx->ev_in[s]) cudaEventDestroy(ctx->ev_in[s]);
        if (ctx->ev_comp[s]) cudaEventDestroy(ctx->ev_comp[s]);
        if (ctx->ev_out[s]) cudaEventDestroy(ctx->ev_out[s]);
    }
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    cudaFree(ctx->d_status);
    delete ctx;
    return QASR_OK;
}

extern "C" const char* qasr_last_error(const qasr_ctx* ctx) { return ctx ? ctx->err : ""; }

extern "C" int qasr_poll_status(qasr_ctx* ctx) {
    if (!ctx) return QASR_ERR_NULL;
    unsigned h = 0;
    QASR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    QASR_CUDA(ctx, cudaMemcpy(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost));
    if (h) QASR_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(h)));
    if (h & QASR_STATUS_TIMEOUT) QASR_FAIL(ctx, QASR_ERR_DEVICE_TIMEOUT, "a device-side wait gave up (status 0x%x)", h);
    if (h & QASR_STATUS_RANGE) QASR_FAIL(ctx, QASR_ERR_RANGE, "a kernel saw a shift outside [1,62] or a negative multiplier");
    return QASR_OK;
}

extern "C" int qasr_set_option(qasr_ctx* ctx, int option, int value) {
    if (!ctx) return QASR_ERR_NULL;
    switch (option) {
        case QASR_OPT_GRAPH: ctx->opt_graph = value != 0; break;
        case QASR_OPT_TENSOR_CORES: ctx->opt_tc = value != 0; break;
        case QASR_OPT_PROFILE: ctx->profiling = value != 0; break;
        case QASR_OPT_SIDE_BRANCH: ctx->opt_side = value != 0; break;
        case QASR_OPT_FRAME_MAJOR_OUTPUT: ctx->opt_dual_out = value != 0; break;
        case QASR_OPT_GEMM_FRAME_TILE:
        case QASR_OPT_DW_FRAME_TILE:
            if (value != 0 && (value < 16 || value > 256 || value % 16 != 0))
                QASR_FAIL(ctx, QASR_ERR_SHAPE, "frame tile %d must be 0 or a multiple of 16 in [16, 256]", value);
            (option == QASR_OPT_GEMM_FRAME_TILE ? ctx->force_gemm_bn : ctx->force_dw_nt) = value;
            break;
        case QASR_OPT_STATIC_WEIGHTS:
            ctx->opt_static_w = value != 0;
            ctx->prepared = false;
            qasr_plan_cache_clear(ctx);
            break;
        default: QASR_FAIL(ctx, QASR_ERR_SHAPE, "unknown option %d", option);
    }
    qasr_plan_cache_clear(ctx);
    return QASR_OK;
}

extern "C" int64_t qasr_launch_count(const qasr_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int qasr_profile_read(qasr_ctx* ctx, qasr_profile_entry* out, int capacity, int* n) {
    if (!ctx || !n) return QASR_ERR_NULL;
    QASR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    *n = (int)ctx->prof.size();
    for (size_t i = 0; i < ctx->prof.size(); ++i) {
        QasrProfRec& r = ctx->prof[i];
        if (out && (int)i < capacity) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, r.e0, r.e1);
            out[i].layer = r.layer; out[i].kernel = r.kernel; out[i].ms = ms; out[i].reserved = 0.f;
            out[i].macs = r.macs; out[i].bytes = r.bytes;
        }
        cudaEventDestroy(r.e0);
        cudaEventDestroy(r.e1);
    }
    ctx->prof.clear();
    return QASR_OK;
}

extern "C" const char* qasr_kernel_name(int kernel) {
    switch (kernel) {
        case QASR_K_DW_GENERIC: return "dw_conv_generic";
        case QASR_K_CONV_GENERIC: return "conv_generic";
        case QASR_K_RESIDUAL_ADD: return "residual_add";
        case QASR_K_DEQUANT: return "dequant";
        case QASR_K_DW_DP4A: return "dw_conv_dp4a";
        case QASR_K_GEMM_TC: return "gemm_i8_tc";
        case QASR_K_CONV_TC: return "conv_i8_tc";
        case QASR_K_GLU: return "glu";
        case QASR_K_CONV_PREP: return "conv_tc_prepare";
        case QASR_K_DW_TC: return "dw_conv_tc";
        default: return "?";
    }
}

// ------------------------------------------------------------------------------------------
// validation helpers
// ------------------------------------------------------------------------------------------
static inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

static int check_conv_params(qasr_ctx* ctx, int B, int C_in, int C_out, int T, int K, int stride,
                             int dilation) {
    if (B <= 0 || C_in <= 0 || C_out <= 0 || T <= 0)
        QASR_FAIL(ctx, QASR_ERR_SHAPE, "sizes must be positive (B=%d C_in=%d C_out=%d T=%d)", B, C_in, C_out, T);
    if (B > 65535) QASR_FAIL(ctx, QASR_ERR_SHAPE, "B=%d exceeds 65535", B);
    if (K < 1 || K > 127 || (K % 2) == 0) QASR_FAIL(ctx, QASR_ERR_SHAPE, "K=%d must be odd and in [1,127]", K);
    if (stride != 1 && stride != 2) QASR_FAIL(ctx, QASR_ERR_SHAPE, "stride=%d must be 1 or 2", stride);
    if (dilation != 1 && dilation != 2) QASR_FAIL(ctx, QASR_ERR_SHAPE, "dilation=%d must be 1 or 2", dilation);
    if ((long long)B * (C_in > C_out ? C_in : C_out) * (long long)T >= (1LL << 40))
        QASR_FAIL(ctx, QASR_ERR_SHAPE, "tensor too large");
    return QASR_OK;
}

static int check_overflow(qasr_ctx* ctx, long long taps, long long max_abs_bias) {
    if (max_abs_bias < 0) QASR_FAIL(ctx, QASR_ERR_SHAPE, "max_abs_bias must be non-negative");
    if (taps * 127LL * 128LL + max_abs_bias >= (1LL << 31))
        QASR_FAIL(ctx, QASR_ERR_OVERFLOW_RISK, "%lld taps with |bias| <= %lld can overflow int32", taps, max_abs_bias);
    return QASR_OK;
}

static int check_rq(qasr_ctx* ctx, qasr_requant rq, const char* what) {
    if (!rq.mult || !rq.shift) QASR_FAIL(ctx, QASR_ERR_NULL, "%s mult/shift is NULL", what);
    if (!aligned(rq.mult, 4)) QASR_FAIL(ctx, QASR_ERR_ALIGN, "%s mult is not 4-byte aligned", what);
    return QASR_OK;
}

static int check_terms_host(qasr_ctx* ctx, int n_terms, const int32_t* mult, const uint8_t* shift, int first) {
    for (int j = first; j < n_terms; ++j) {
        if (mult[j] < 0 || shift[j] < 1 || shift[j] > 62)
            QASR_FAIL(ctx, QASR_ERR_RANGE, "term %d: mult=%d shift=%d out of range", j, mult[j], (int)shift[j]);
    }
    return QASR_OK;
}

// ------------------------------------------------------------------------------------------
// dispatch (the only place that picks a kernel)
// ------------------------------------------------------------------------------------------
static int run_dw(qasr_ctx* ctx, const QasrDwArgs& a) {
    int used = qasr_try_dw_fast(ctx, a);
    if (used < 0) return used;
    if (!used) {
        QasrLaunchScope ls(ctx, QASR_K_DW_GENERIC, qasr_dw_macs(a), qasr_dw_bytes(a));
        QASR_CUDA(ctx, qasr_launch_dw_generic(a, ctx->d_status, ctx->stream));
    }
    return QASR_OK;
}

static int run_conv(qasr_ctx* ctx, const QasrConvArgs& a) {
    int used = qasr_try_conv_tc(ctx, a);
    if (used < 0) return used;
    if (!used) {
        QasrLaunchScope ls(ctx, QASR_K_CONV_GENERIC, qasr_conv_macs(a), qasr_conv_bytes(a));
        QASR_CUDA(ctx, qasr_launch_conv_generic(a, ctx->d_status, ctx->stream));
    }
    return QASR_OK;
}

// The constant arrays a convolution / depthwise launch reads.
static QasrPrefetch conv_constants(const QasrConvArgs& a) {
    QasrPrefetch pf;
    memset(&pf, 0, sizeof(pf));
    pf.ptr[0] = a.w;     pf.bytes[0] = (uint32_t)((size_t)a.C_out * a.C_in * a.K);
    pf.ptr[1] = a.bias;  pf.bytes[1] = (uint32_t)(a.C_out * 4);
    pf.ptr[2] = a.mult;  pf.bytes[2] = (uint32_t)(a.C_out * 4);
    pf.ptr[3] = a.shift; pf.bytes[3] = (uint32_t)a.C_out;
    return pf;
}
static QasrPrefetch dw_constants(const int8_t* w, const int32_t* mult, const uint8_t* shift, int C, int K) {
    QasrPrefetch pf;
    memset(&pf, 0, sizeof(pf));
    pf.ptr[0] = w;     pf.bytes[0] = (uint32_t)(C * K);
    pf.ptr[1] = mult;  pf.bytes[1] = (uint32_t)(C * 4);
    pf.ptr[2] = shift; pf.bytes[2] = (uint32_t)C;
    return pf;
}

static int run_tcs(qasr_ctx* ctx, const QasrDwArgs& d, QasrConvArgs p, void* scratch) {
    QasrDwArgs d2 = d;
    d2.y = (int8_t*)scratch;
    p.x = (const int8_t*)scratch;
    const QasrPrefetch after = ctx->prefetch;       // what follows the block: the pointwise kernel's hint
    ctx->prefetch = conv_constants(p);              // the depthwise kernel fetches the pointwise constants
    int rc = run_dw(ctx, d2);
    ctx->prefetch = after;
    if (rc != QASR_OK) return rc;
    return run_conv(ctx, p);
}

// ------------------------------------------------------------------------------------------
// single operations
// ------------------------------------------------------------------------------------------
extern "C" int qasr_dw_conv(qasr_ctx* ctx, const int8_t* x, int B, int C, int T,
                            const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                            int8_t* y) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x || !w_dw || !y) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_dw_conv: NULL tensor");
    int rc = check_conv_params(ctx, B, C, C, T, K, stride, dilation);
    if (rc) return rc;
    if (C > 65535) QASR_FAIL(ctx, QASR_ERR_SHAPE, "C=%d exceeds 65535", C);
    if ((rc = check_rq(ctx, rq_dw, "rq_dw"))) return rc;
    if ((rc = check_overflow(ctx, K, 0))) return rc;
    if ((const void*)x == (const void*)y) QASR_FAIL(ctx, QASR_ERR_ALIAS, "qasr_dw_conv: y aliases x");
    QasrDwArgs a{x, w_dw, rq_dw.mult, rq_dw.shift, y, B, C, T, (T - 1) / stride + 1, K, stride, dilation};
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    return run_dw(ctx, a);
}

static int fill_terms(qasr_ctx* ctx, QasrTerms& t, int n_terms, const int8_t* const* terms,
                      const int32_t* mult, const uint8_t* shift, bool conv_epilogue, const void* y) {
    t.n = 0;
    if (n_terms == 0 && conv_epilogue) return QASR_OK;
    const int lo = conv_epilogue ? 2 : 1;
    if (n_terms < lo || n_terms > QASR_MAX_TERMS)
        QASR_FAIL(ctx, QASR_ERR_SHAPE, "n_terms=%d must be %s%d..%d", n_terms, conv_epilogue ? "0 or " : "", lo, QASR_MAX_TERMS);
    if (!terms || !mult || !shift) QASR_FAIL(ctx, QASR_ERR_NULL, "terms/mult/shift is NULL");
    int rc = check_terms_host(ctx, n_terms, mult, shift, 0);
    if (rc) return rc;
    t.n = n_terms;
    for (int j = 0; j < n_terms; ++j) {
        t.ptr[j] = (conv_epilogue && j == 0) ? nullptr : terms[j];
        if (!(conv_epilogue && j == 0)) {
            if (!terms[j]) QASR_FAIL(ctx, QASR_ERR_NULL, "term %d is NULL", j);
            if ((const void*)terms[j] == y) QASR_FAIL(ctx, QASR_ERR_ALIAS, "y aliases term %d", j);
        }
        t.mult[j] = mult[j];
        t.shift[j] = shift[j];
    }
    return QASR_OK;
}

extern "C" int qasr_conv(qasr_ctx* ctx, const int8_t* x, int B, int C_in, int T,
                         const int8_t* w, int C_out, int K, int stride, int dilation,
                         const int32_t* bias, int32_t max_abs_bias, qasr_requant rq, int relu,
                         int n_terms, const int8_t* const* terms, const int32_t* term_mult,
                         const uint8_t* term_shift, int8_t* y, int32_t* y_int32) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x || !w || (!y && !y_int32)) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_conv: NULL tensor");
    int rc = check_conv_params(ctx, B, C_in, C_out, T, K, stride, dilation);
    if (rc) return rc;
    if (C_out > 65535 * 64) QASR_FAIL(ctx, QASR_ERR_SHAPE, "C_out too large");
    if (!y_int32 && (rc = check_rq(ctx, rq, "rq"))) return rc;
    if (bias && !aligned(bias, 4)) QASR_FAIL(ctx, QASR_ERR_ALIGN, "bias is not 4-byte aligned");
    if (y_int32 && !aligned(y_int32, 4)) QASR_FAIL(ctx, QASR_ERR_ALIGN, "y_int32 is not 4-byte aligned");
    if ((rc = check_overflow(ctx, (long long)C_in * K, bias ? max_abs_bias : 0))) return rc;
    if ((const void*)x == (const void*)y || (const void*)x == (const void*)y_int32)
        QASR_FAIL(ctx, QASR_ERR_ALIAS, "qasr_conv: output aliases x");
    QasrConvArgs a;
    memset(&a, 0, sizeof(a));
    a.x = x; a.w = w; a.bias = bias; a.mult = rq.mult; a.shift = rq.shift;
    a.y = y_int32 ? nullptr : y; a.y_int32 = y_int32;
    a.B = B; a.C_in = C_in; a.C_out = C_out; a.T = T; a.T_out = (T - 1) / stride + 1;
    a.K = K; a.stride = stride; a.dilation = dilation; a.relu = relu ? 1 : 0;
    if (y_int32 && n_terms != 0) QASR_FAIL(ctx, QASR_ERR_SHAPE, "residual terms cannot be combined with int32 output");
    if ((rc = fill_terms(ctx, a.terms, n_terms, terms, term_mult, term_shift, true, y))) return rc;
    a.scratch = ctx->conv_scratch;
    a.scratch_bytes = ctx->conv_scratch_bytes;
    if (a.scratch) {
        const char* lo = (const char*)a.scratch;
        const char* hi = lo + a.scratch_bytes;
        auto inside = [&](const void* q) { return q && (const char*)q >= lo && (const char*)q < hi; };
        if (inside(x) || inside(y) || inside(y_int32) || inside(w)) QASR_FAIL(ctx, QASR_ERR_ALIAS, "qasr_conv: a tensor lies inside the lent scratch");
    }
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    return run_conv(ctx, a);
}

extern "C" int qasr_conv_scratch_bytes(int B, int C_in, int C_out, int T, int K, int stride, size_t* bytes) {
    if (!bytes) return QASR_ERR_NULL;
    if (B <= 0 || C_in <= 0 || C_out <= 0 || T <= 0 || K < 1 || (K % 2) == 0 || K > 127 || (stride != 1 && stride != 2))
        return QASR_ERR_SHAPE;
    *bytes = qasr_conv_tc_scratch_bytes(B, C_in, C_out, T, K, stride);
    return QASR_OK;
}

extern "C" int qasr_set_conv_scratch(qasr_ctx* ctx, void* scratch, size_t bytes) {
    if (!ctx) return QASR_ERR_NULL;
    if ((scratch == nullptr) != (bytes == 0)) QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_set_conv_scratch: pointer and size must both be given or both be zero");
    if (scratch && !aligned(scratch, 256)) QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_set_conv_scratch: scratch is not 256-byte aligned");
    ctx->conv_scratch = scratch;
    ctx->conv_scratch_bytes = bytes;
    return QASR_OK;
}

extern "C" int qasr_tcs_block_workspace_bytes(int B, int C_in, int C_out, int T, int K, int stride,
                                              int dilation, size_t* bytes) {
    if (!bytes) return QASR_ERR_NULL;
    if (B <= 0 || C_in <= 0 || C_out <= 0 || T <= 0 || K < 1 || (K % 2) == 0 || K > 127 ||
        (stride != 1 && stride != 2) || (dilation != 1 && dilation != 2))
        return QASR_ERR_SHAPE;
    const size_t t_out = (size_t)(T - 1) / stride + 1;
    *bytes = ((size_t)B * C_in * t_out + 255) / 256 * 256;  // the depthwise output
    return QASR_OK;
}

extern "C" int qasr_tcs_block(qasr_ctx* ctx, const int8_t* x, int B, int C_in, int T,
                              const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                              const int8_t* w_pw, int C_out, const int32_t* bias, int32_t max_abs_bias,
                              qasr_requant rq_pw, int relu, int8_t* y,
                              void* workspace, size_t workspace_bytes) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x || !w_dw || !w_pw || !y) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_tcs_block: NULL tensor");
    int rc = check_conv_params(ctx, B, C_in, C_out, T, K, stride, dilation);
    if (rc) return rc;
    if (C_in > 65535) QASR_FAIL(ctx, QASR_ERR_SHAPE, "C_in=%d exceeds 65535", C_in);
    if ((rc = check_rq(ctx, rq_dw, "rq_dw")) || (rc = check_rq(ctx, rq_pw, "rq_pw"))) return rc;
    if (bias && !aligned(bias, 4)) QASR_FAIL(ctx, QASR_ERR_ALIGN, "bias is not 4-byte aligned");
    if ((rc = check_overflow(ctx, K, 0)) || (rc = check_overflow(ctx, C_in, bias ? max_abs_bias : 0))) return rc;
    if ((const void*)x == (const void*)y) QASR_FAIL(ctx, QASR_ERR_ALIAS, "qasr_tcs_block: y aliases x");
    size_t need = 0;
    qasr_tcs_block_workspace_bytes(B, C_in, C_out, T, K, stride, dilation, &need);
    if (need && (!workspace || workspace_bytes < need || !aligned(workspace, 256)))
        QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_tcs_block needs %zu bytes of 256-byte aligned workspace", need);
    if (workspace == (void*)x || workspace == (void*)y) QASR_FAIL(ctx, QASR_ERR_ALIAS, "workspace aliases a tensor");
    const int T_out = (T - 1) / stride + 1;
    QasrDwArgs d{x, w_dw, rq_dw.mult, rq_dw.shift, nullptr, B, C_in, T, T_out, K, stride, dilation};
    QasrConvArgs p;
    memset(&p, 0, sizeof(p));
    p.w = w_pw; p.bias = bias; p.mult = rq_pw.mult; p.shift = rq_pw.shift; p.y = y;
    p.B = B; p.C_in = C_in; p.C_out = C_out; p.T = T_out; p.T_out = T_out; p.K = 1; p.stride = 1; p.dilation = 1;
    p.relu = relu ? 1 : 0;
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    return run_tcs(ctx, d, p, workspace);
}

extern "C" int qasr_residual_requant_add(qasr_ctx* ctx, int n_terms, const int8_t* const* terms,
                                         const int32_t* mult, const uint8_t* shift,
                                         int B, int C, int T, int relu, int8_t* y) {
    if (!ctx) return QASR_ERR_NULL;
    if (!y) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_residual_requant_add: y is NULL");
    if (B <= 0 || C <= 0 || T <= 0) QASR_FAIL(ctx, QASR_ERR_SHAPE, "sizes must be positive");
    QasrTerms t;
    memset(&t, 0, sizeof(t));
    int rc = fill_terms(ctx, t, n_terms, terms, mult, shift, false, y);
    if (rc) return rc;
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    {
        QasrLaunchScope ls(ctx, QASR_K_RESIDUAL_ADD, 0, (double)B * C * T * (n_terms + 1));
        QASR_CUDA(ctx, qasr_launch_residual_add(t, (size_t)B * C * T, relu ? 1 : 0, y, ctx->d_status, ctx->stream));
    }
    return QASR_OK;
}

extern "C" int qasr_dequant_logits(qasr_ctx* ctx, const int32_t* acc, int B, int C, int T,
                                   const float* scale, float* out) {
    if (!ctx) return QASR_ERR_NULL;
    if (!acc || !scale || !out) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_dequant_logits: NULL pointer");
    if (B <= 0 || C <= 0 || T <= 0) QASR_FAIL(ctx, QASR_ERR_SHAPE, "sizes must be positive");
    if (!aligned(acc, 4) || !aligned(scale, 4) || !aligned(out, 4)) QASR_FAIL(ctx, QASR_ERR_ALIGN, "4-byte alignment required");
    if ((const void*)acc == (const void*)out) QASR_FAIL(ctx, QASR_ERR_ALIAS, "out aliases acc");
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    {
        QasrLaunchScope ls(ctx, QASR_K_DEQUANT, 0, (double)B * C * T * 8);
        QASR_CUDA(ctx, qasr_launch_dequant(acc, B, C, T, scale, out, ctx->stream));
    }
    return QASR_OK;
}

extern "C" int qasr_glu(qasr_ctx* ctx, const int8_t* x, int B, int C, int T, int q_c, qasr_requant rq, int8_t* y) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x || !y) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_glu: NULL tensor");
    if (B <= 0 || C <= 0 || T <= 0 || q_c < 1 || q_c > 128) QASR_FAIL(ctx, QASR_ERR_SHAPE, "qasr_glu: bad sizes or q_c");
    int rc = check_rq(ctx, rq, "rq");
    if (rc) return rc;
    if ((const void*)x == (const void*)y) QASR_FAIL(ctx, QASR_ERR_ALIAS, "qasr_glu: y aliases x");
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    {
        QasrLaunchScope ls(ctx, QASR_K_GLU, 0, (double)B * C * T * 3);
        QASR_CUDA(ctx, qasr_launch_glu(x, B, C, T, q_c, rq.mult, rq.shift, y, ctx->d_status, ctx->stream));
    }
    return QASR_OK;
}

// ------------------------------------------------------------------------------------------
// layer table: validation + buffer plan
// ------------------------------------------------------------------------------------------
namespace {

constexpr int kMaxBufs = 4096;

struct BufState {
    int C = 0, T = 0;       // shape last written
    size_t bytes = 0;       // largest tensor ever written
    size_t offset = 0;
    bool live = false;
};

struct TablePlan {
    std::vector<BufState> bufs;   // index = buffer id; 0 = encoder input
    std::vector<int> t_in, t_out; // per layer
    size_t scratch_offset = 0, scratch_bytes = 0;
    // second home of a frame-major input copy: a K-tap convolution reads its own copy from one region while its
    // epilogue writes the next K-tap convolution's copy into the other
    size_t scratch2_offset = 0, scratch2_bytes = 0;
    std::vector<size_t> wt_offset;   // per layer: home of its regrouped weights (implicit-GEMM path), or SIZE_MAX
    size_t total = 0;
    int C_last = 0, T_last = 0;
};

#define PLAN_FAIL(code, ...)                        \
    do {                                            \
        if (err) snprintf(err, errlen, __VA_ARGS__); \
        return (code);                              \
    } while (0)

int plan_table(const qasr_layer* tb, int n, int B, int C_in, int T, TablePlan& p, char* err, size_t errlen) {
    if (!tb) PLAN_FAIL(QASR_ERR_NULL, "layer table is NULL");
    if (n <= 0 || B <= 0 || C_in <= 0 || T <= 0) PLAN_FAIL(QASR_ERR_SHAPE, "n_layers, B, C_in, T must be positive");
    if (B > 65535) PLAN_FAIL(QASR_ERR_SHAPE, "B exceeds 65535");
    p.bufs.assign(1, BufState());
    p.bufs[0].C = C_in;
    p.bufs[0].T = T;
    p.bufs[0].live = true;
    p.t_in.assign(n, 0);
    p.t_out.assign(n, 0);
    p.wt_offset.assign(n, SIZE_MAX);
    size_t wt_total = 0;
    for (int li = 0; li < n; ++li) {
        const qasr_layer& L = tb[li];
        const bool last = li == n - 1;
        if (L.kind < QASR_LAYER_DW || L.kind > QASR_LAYER_GLU) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: unknown kind %d", li, L.kind);
        if (L.out_buf < 1 || L.out_buf >= kMaxBufs) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: out_buf %d out of range", li, L.out_buf);
        if ((L.out_int32 != 0) != last) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: exactly the last layer must have out_int32 set", li);
        int C_o, T_i, T_o;
        if (L.kind == QASR_LAYER_ADD) {
            if (L.n_terms < 1 || L.n_terms > QASR_MAX_TERMS) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: n_terms %d", li, L.n_terms);
            if (L.out_int32) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: an add cannot produce the int32 logits", li);
            for (int j = 0; j < L.n_terms; ++j) {
                const int bid = L.term_buf[j];
                if (bid < 0 || bid >= (int)p.bufs.size() || !p.bufs[bid].live) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: term buffer %d not written yet", li, bid);
                if (bid == L.out_buf) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: out_buf aliases term %d", li, j);
                if (p.bufs[bid].C != p.bufs[L.term_buf[0]].C || p.bufs[bid].T != p.bufs[L.term_buf[0]].T)
                    PLAN_FAIL(QASR_ERR_TABLE, "layer %d: term %d shape mismatch", li, j);
                if (L.term_mult[j] < 0 || L.term_shift[j] < 1 || L.term_shift[j] > 62) PLAN_FAIL(QASR_ERR_RANGE, "layer %d: term %d constants out of range", li, j);
            }
            C_o = p.bufs[L.term_buf[0]].C;
            T_i = T_o = p.bufs[L.term_buf[0]].T;
        } else if (L.kind == QASR_LAYER_GLU) {
            if (L.in_buf < 0 || L.in_buf >= (int)p.bufs.size() || !p.bufs[L.in_buf].live) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: in_buf %d not written yet", li, L.in_buf);
            if (L.in_buf == L.out_buf) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: out_buf equals in_buf", li);
            if (L.C_out <= 0 || L.C_in != 2 * L.C_out || L.C_in != p.bufs[L.in_buf].C) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: a GLU halves the channel count of its input", li);
            if (L.glu_qc < 1 || L.glu_qc > 128) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: glu_qc %d must be in [1,128]", li, L.glu_qc);
            if (!L.rq.mult || !L.rq.shift) PLAN_FAIL(QASR_ERR_NULL, "layer %d: rq is NULL", li);
            if (!aligned(L.rq.mult, 4)) PLAN_FAIL(QASR_ERR_ALIGN, "layer %d: rq.mult misaligned", li);
            if (L.n_terms != 0 || L.out_int32) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: a GLU takes no residual terms and gives int8", li);
            C_o = L.C_out;
            T_i = T_o = p.bufs[L.in_buf].T;
        } else {
            if (L.in_buf < 0 || L.in_buf >= (int)p.bufs.size() || !p.bufs[L.in_buf].live) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: in_buf %d not written yet", li, L.in_buf);
            if (L.in_buf == L.out_buf) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: out_buf equals in_buf", li);
            if (L.C_in <= 0 || L.C_out <= 0) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: channel counts must be positive", li);
            if (L.C_in != p.bufs[L.in_buf].C) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: C_in %d but buffer %d holds %d channels", li, L.C_in, L.in_buf, p.bufs[L.in_buf].C);
            if (L.K < 1 || L.K > 127 || (L.K % 2) == 0) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: K=%d must be odd and in [1,127]", li, L.K);
            if ((L.stride != 1 && L.stride != 2) || (L.dilation != 1 && L.dilation != 2)) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: stride/dilation must be 1 or 2", li);
            if (L.kind == QASR_LAYER_PW && (L.K != 1 || L.stride != 1 || L.dilation != 1)) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: a pointwise layer has K=stride=dilation=1", li);
            if (L.kind == QASR_LAYER_DW && L.C_in != L.C_out) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: depthwise needs C_in == C_out", li);
            if (L.C_in > 65535 && (L.kind == QASR_LAYER_DW || L.kind == QASR_LAYER_TCS)) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: too many depthwise channels", li);
            const bool has_dw = L.kind == QASR_LAYER_DW || L.kind == QASR_LAYER_TCS;
            const bool has_mm = L.kind != QASR_LAYER_DW;
            if (has_dw) {
                if (!L.w_dw || !L.rq_dw.mult || !L.rq_dw.shift) PLAN_FAIL(QASR_ERR_NULL, "layer %d: depthwise constants are NULL", li);
                if (!aligned(L.rq_dw.mult, 4)) PLAN_FAIL(QASR_ERR_ALIGN, "layer %d: rq_dw.mult misaligned", li);
                if ((long long)L.K * 127 * 128 >= (1LL << 31)) PLAN_FAIL(QASR_ERR_OVERFLOW_RISK, "layer %d", li);
            }
            if (has_mm) {
                if (!L.w) PLAN_FAIL(QASR_ERR_NULL, "layer %d: w is NULL", li);
                if (!L.out_int32 && (!L.rq.mult || !L.rq.shift)) PLAN_FAIL(QASR_ERR_NULL, "layer %d: rq is NULL", li);
                if ((L.rq.mult && !aligned(L.rq.mult, 4)) || (L.bias && !aligned(L.bias, 4))) PLAN_FAIL(QASR_ERR_ALIGN, "layer %d: int32 constants misaligned", li);
                if (L.max_abs_bias < 0) PLAN_FAIL(QASR_ERR_SHAPE, "layer %d: max_abs_bias negative", li);
                const long long taps = (long long)L.C_in * (L.kind == QASR_LAYER_DENSE ? L.K : 1);
                if (taps * 127LL * 128LL + (L.bias ? L.max_abs_bias : 0) >= (1LL << 31))
                    PLAN_FAIL(QASR_ERR_OVERFLOW_RISK, "layer %d: %lld taps can overflow int32", li, taps);
            }
            T_i = p.bufs[L.in_buf].T;
            T_o = (L.kind == QASR_LAYER_PW) ? T_i : (T_i - 1) / L.stride + 1;
            C_o = L.C_out;
            if (L.n_terms != 0) {
                if (!has_mm || L.out_int32) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: residual terms need an int8 conv output", li);
                if (L.n_terms < 2 || L.n_terms > QASR_MAX_TERMS) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: n_terms %d", li, L.n_terms);
                for (int j = 0; j < L.n_terms; ++j) {
                    if (L.term_mult[j] < 0 || L.term_shift[j] < 1 || L.term_shift[j] > 62) PLAN_FAIL(QASR_ERR_RANGE, "layer %d: term %d constants out of range", li, j);
                    if (j == 0) continue;
                    const int bid = L.term_buf[j];
                    if (bid < 0 || bid >= (int)p.bufs.size() || !p.bufs[bid].live) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: term buffer %d not written yet", li, bid);
                    if (bid == L.out_buf) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: out_buf aliases term %d", li, j);
                    if (p.bufs[bid].C != C_o || p.bufs[bid].T != T_o) PLAN_FAIL(QASR_ERR_TABLE, "layer %d: term %d has shape [%d][%d], expected [%d][%d]", li, j, p.bufs[bid].C, p.bufs[bid].T, C_o, T_o);
                }
            }
            if (L.kind == QASR_LAYER_TCS) {
                const size_t sb = (size_t)B * L.C_in * T_o;
                if (sb > p.scratch_bytes) p.scratch_bytes = sb;
            } else if ((L.kind == QASR_LAYER_DENSE || L.kind == QASR_LAYER_PW) &&
                       !qasr_conv_shape_fits_gemm(L.C_in, L.K, L.stride, L.dilation, T_o)) {
                // implicit-GEMM path: the frame-major input copy shares the scratch region, the regrouped
                // weights get a place of their own so that they can outlive the call
                const size_t sb = qasr_conv_tc_input_bytes(B, L.C_in, T_i, L.stride);
                if (sb > p.scratch_bytes) p.scratch_bytes = sb;
                if (L.stride == 1 && sb > p.scratch2_bytes) p.scratch2_bytes = sb;
                p.wt_offset[li] = wt_total;
                wt_total += qasr_conv_tc_weight_bytes(L.C_in, L.C_out, L.K);
            }
        }
        p.t_in[li] = T_i;
        p.t_out[li] = T_o;
        if (last) {
            p.C_last = C_o;
            p.T_last = T_o;
        } else {
            if ((int)p.bufs.size() <= L.out_buf) p.bufs.resize(L.out_buf + 1);
            BufState& ob = p.bufs[L.out_buf];
            ob.C = C_o;
            ob.T = T_o;
            ob.live = true;
            const size_t bytes = (size_t)B * C_o * T_o;
            if (bytes > ob.bytes) ob.bytes = bytes;
        }
    }
    size_t off = 0;
    for (size_t i = 1; i < p.bufs.size(); ++i) {
        p.bufs[i].offset = off;
        off += (p.bufs[i].bytes + 255) / 256 * 256;
    }
    p.scratch_offset = off;
    off += (p.scratch_bytes + 255) / 256 * 256;
    p.scratch2_offset = off;
    off += (p.scratch2_bytes + 255) / 256 * 256;
    for (int li = 0; li < n; ++li)
        if (p.wt_offset[li] != SIZE_MAX) p.wt_offset[li] += off;
    off += wt_total;
    p.total = off;
    return QASR_OK;
}

struct Staging { size_t x, lq, lf, total; };
Staging staging_for(const TablePlan& p, int B, int C_in, int T) {
    Staging s;
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    s.x = 0;
    s.lq = up((size_t)B * C_in * T);
    s.lf = s.lq + up((size_t)B * p.C_last * p.T_last * 4);
    s.total = s.lf + up((size_t)B * p.C_last * p.T_last * 4);
    return s;
}

}  // namespace

extern "C" size_t qasr_layer_size(void) { return sizeof(qasr_layer); }

extern "C" int qasr_encoder_workspace_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                            size_t* bytes) {
    if (!bytes) return QASR_ERR_NULL;
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, nullptr, 0);
    if (rc) return rc;
    *bytes = p.total;
    return QASR_OK;
}

extern "C" int qasr_encoder_buffer_info(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                        int buf_id, size_t* offset, int* C, int* T_len) {
    if (!offset || !C || !T_len) return QASR_ERR_NULL;
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, nullptr, 0);
    if (rc) return rc;
    if (buf_id < 1 || buf_id >= (int)p.bufs.size() || !p.bufs[buf_id].live) return QASR_ERR_TABLE;
    *offset = p.bufs[buf_id].offset;
    *C = p.bufs[buf_id].C;
    *T_len = p.bufs[buf_id].T;
    return QASR_OK;
}

extern "C" int qasr_encoder_host_staging_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                               size_t* bytes) {
    if (!bytes) return QASR_ERR_NULL;
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, nullptr, 0);
    if (rc) return rc;
    *bytes = staging_for(p, B, C_in, T).total;
    return QASR_OK;
}

// Enqueue every layer of a validated table (no graph handling here).
static int enqueue_table(qasr_ctx* ctx, const qasr_layer* tb, int n, const TablePlan& p,
                         const int8_t* x, int B, char* ws, int32_t* logits_q, float* logits,
                         const float* out_scale, bool weights_ready = false, bool capturing = false) {
    auto buf_ptr = [&](int id) -> int8_t* { return id == 0 ? const_cast<int8_t*>(x) : (int8_t*)(ws + p.bufs[id].offset); };
    // Shapes of buffers change as layers overwrite them, so they are re-tracked here.
    std::vector<int> curC(p.bufs.size(), 0);
    curC[0] = p.bufs[0].C;
    // Side branch (only while the table is being captured into a graph): a pointwise convolution whose result
    // the next layer does not read -- a block's residual projection; several in a row for dense residuals -- runs
    // on a second stream with a small grid, on the SMs that the main chain's 128-item kernels leave idle, and joins
    // the main chain in front of the first layer that reads one of its outputs or overwrites one of its tensors.
    // While a branch is pending the main chain's persistent kernels launch 128 CTAs (their item counts are
    // multiples of 128 at these shapes anyway). The branch's kernels follow one another in stream order.
    struct {
        bool pending = false;
        std::vector<int> in_bufs, out_bufs;      // tensors the pending branch reads / writes
        bool reads(int b) const { for (int v : in_bufs) if (v == b) return true; return false; }
        bool writes(int b) const { for (int v : out_bufs) if (v == b) return true; return false; }
    } side;
    // Frame-major copy of a tensor that a K-tap convolution's epilogue has already left in one of the two scratch
    // regions (buffer id, region), valid until that buffer or that region is written again.
    int ft_buf = -1, ft_region = 0;
    auto scratch_region = [&](int r, size_t& bytes) -> char* {
        bytes = r ? p.scratch2_bytes : p.scratch_bytes;
        return ws + (r ? p.scratch2_offset : p.scratch_offset);
    };
    // A layer that takes the scratch-using convolution path (anything the pointwise GEMM does not take).
    auto wants_scratch = [&](const qasr_layer& Q, int T_out) {
        return (Q.kind == QASR_LAYER_DENSE || Q.kind == QASR_LAYER_PW) &&
               !qasr_conv_shape_fits_gemm(Q.C_in, Q.K, Q.stride, Q.dilation, T_out);
    };
    const int main_slots = 128;
    const bool side_ok = capturing && ctx->opt_side && ctx->opt_tc && ctx->encode_tiled && !ctx->profiling &&
                         ctx->sm_count >= main_slots + 16;
    auto join_side = [&]() -> int {
        if (!side.pending) return QASR_OK;
        QASR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_side, 0));
        side.pending = false;
        side.in_bufs.clear();
        side.out_bufs.clear();
        ctx->grid_cap = 0;
        return QASR_OK;
    };
    for (int li = 0; li < n; ++li) {
        const qasr_layer& L = tb[li];
        const int T_i = p.t_in[li], T_o = p.t_out[li];
        int rc = QASR_OK;
        ctx->cur_layer = li;
        // Does this layer go to the side branch? A pointwise layer on the tensor-core GEMM path whose output the
        // next layer neither reads nor overwrites, while the main chain's kernels fit 128 CTAs.
        bool to_side = false;
        if (side_ok && L.kind == QASR_LAYER_PW && !L.out_int32 && L.n_terms == 0 && li + 2 < n &&
            qasr_conv_shape_fits_gemm(L.C_in, 1, 1, 1, T_o) && (long long)B * ((T_o + 207) / 208) <= main_slots) {
            const qasr_layer& N = tb[li + 1];
            bool next_reads = N.kind != QASR_LAYER_ADD && N.in_buf == L.out_buf;
            for (int j = (N.kind == QASR_LAYER_ADD ? 0 : 1); j < N.n_terms; ++j)
                if (N.term_buf[j] == L.out_buf) next_reads = true;
            to_side = !next_reads && N.out_buf != L.out_buf && N.out_buf != L.in_buf;
        }
        if (side.pending && !to_side) {
            // join in front of a main-chain layer that reads one of the branch's outputs or writes one of its
            // tensors (a layer that itself joins the branch follows the pending kernels in stream order)
            bool hazard = side.reads(L.out_buf) || side.writes(L.out_buf) || L.out_int32;
            if (L.kind != QASR_LAYER_ADD && side.writes(L.in_buf)) hazard = true;
            for (int j = (L.kind == QASR_LAYER_ADD ? 0 : 1); j < L.n_terms; ++j)
                if (side.writes(L.term_buf[j])) hazard = true;
            if (hazard && (rc = join_side())) return rc;
        }
        if (!L.out_int32 && L.out_buf == ft_buf) ft_buf = -1;     // the tensor is overwritten: its copy is stale
        if (L.kind == QASR_LAYER_ADD) {
            QasrTerms t;
            memset(&t, 0, sizeof(t));
            t.n = L.n_terms;
            for (int j = 0; j < L.n_terms; ++j) {
                t.ptr[j] = buf_ptr(L.term_buf[j]);
                t.mult[j] = L.term_mult[j];
                t.shift[j] = L.term_shift[j];
            }
            const int C = curC[L.term_buf[0]];
            {
                QasrLaunchScope ls(ctx, QASR_K_RESIDUAL_ADD, 0, (double)B * C * T_o * (L.n_terms + 1));
                QASR_CUDA(ctx, qasr_launch_residual_add(t, (size_t)B * C * T_o, L.relu ? 1 : 0, buf_ptr(L.out_buf), ctx->d_status, ctx->stream));
            }
            curC[L.out_buf] = C;
            continue;
        }
        const int8_t* in = buf_ptr(L.in_buf);
        // the constants of the layer that follows, for the last kernel of this one to ask the L2 for
        memset(&ctx->prefetch, 0, sizeof(ctx->prefetch));
        if (li + 1 < n) {
            const qasr_layer& N = tb[li + 1];
            if (N.kind == QASR_LAYER_TCS || N.kind == QASR_LAYER_DW) {
                ctx->prefetch = dw_constants(N.w_dw, N.rq_dw.mult, N.rq_dw.shift, N.C_in, N.K);
            } else if (N.kind == QASR_LAYER_PW || N.kind == QASR_LAYER_DENSE) {
                QasrConvArgs na;
                memset(&na, 0, sizeof(na));
                na.w = N.w; na.bias = N.bias; na.mult = N.rq.mult; na.shift = N.rq.shift;
                na.C_in = N.C_in; na.C_out = N.C_out; na.K = N.K;
                ctx->prefetch = conv_constants(na);
            }
        }
        if (L.kind == QASR_LAYER_GLU) {
            QasrLaunchScope ls(ctx, QASR_K_GLU, 0, (double)B * L.C_out * T_o * 3);
            QASR_CUDA(ctx, qasr_launch_glu(in, B, L.C_out, T_o, L.glu_qc, L.rq.mult, L.rq.shift, buf_ptr(L.out_buf), ctx->d_status, ctx->stream,
                                           ctx->opt_pdl ? 1 : 0));
            curC[L.out_buf] = L.C_out;
            continue;
        }
        if (L.kind == QASR_LAYER_DW) {
            QasrDwArgs d{in, L.w_dw, L.rq_dw.mult, L.rq_dw.shift, buf_ptr(L.out_buf), B, L.C_in, T_i, T_o, L.K, L.stride, L.dilation};
            rc = run_dw(ctx, d);
        } else {
            QasrConvArgs a;
            memset(&a, 0, sizeof(a));
            a.x = in; a.w = L.w; a.bias = L.bias; a.mult = L.rq.mult; a.shift = L.rq.shift;
            a.B = B; a.C_in = L.C_in; a.C_out = L.C_out; a.relu = L.relu ? 1 : 0;
            if (L.out_int32) a.y_int32 = logits_q; else a.y = buf_ptr(L.out_buf);
            a.terms.n = L.n_terms;
            for (int j = 0; j < L.n_terms; ++j) {
                a.terms.ptr[j] = j == 0 ? nullptr : buf_ptr(L.term_buf[j]);
                a.terms.mult[j] = L.term_mult[j];
                a.terms.shift[j] = L.term_shift[j];
            }
            if (to_side) {
                if (!ctx->side_stream) QASR_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking));
                if (!ctx->ev_fork) QASR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
                if (!ctx->ev_side) QASR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_side, cudaEventDisableTiming));
                a.T = T_i; a.T_out = T_o; a.K = 1; a.stride = 1; a.dilation = 1;
                QASR_CUDA(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
                QASR_CUDA(ctx, cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0));
                cudaStream_t main_stream = ctx->stream;
                ctx->stream = ctx->side_stream;
                ctx->grid_cap = ctx->sm_count - main_slots;
                rc = run_conv(ctx, a);
                ctx->stream = main_stream;
                ctx->grid_cap = main_slots;
                if (rc) return rc;
                QASR_CUDA(ctx, cudaEventRecord(ctx->ev_side, ctx->side_stream));
                side.pending = true;
                side.in_bufs.push_back(L.in_buf);
                side.out_bufs.push_back(L.out_buf);
            } else if (L.kind == QASR_LAYER_TCS) {
                QasrDwArgs d{in, L.w_dw, L.rq_dw.mult, L.rq_dw.shift, nullptr, B, L.C_in, T_i, T_o, L.K, L.stride, L.dilation};
                a.T = T_o; a.T_out = T_o; a.K = 1; a.stride = 1; a.dilation = 1;
                if (ft_region == 0) ft_buf = -1;        // the depthwise output goes to the first scratch region
                rc = run_tcs(ctx, d, a, ws + p.scratch_offset);
            } else {
                a.T = T_i; a.T_out = T_o; a.K = L.K; a.stride = L.stride; a.dilation = L.dilation;
                // the frame-major input copy: where the producing layer left it, else region 0 (transposed there)
                int in_region = 0;
                if (wants_scratch(L, T_o)) {
                    if (ft_buf == L.in_buf && L.stride == 1) {
                        in_region = ft_region;
                        a.xt_ready = 1;
                    } else if (ft_region == 0) {
                        ft_buf = -1;
                    }
                }
                a.scratch = scratch_region(in_region, a.scratch_bytes);
                if (p.wt_offset[li] != SIZE_MAX) {
                    a.wt = ws + p.wt_offset[li];
                    a.wt_ready = weights_ready ? 1 : 0;
                }
                // Second, frame-major output for the K-tap convolution that reads this tensor next: the first
                // scratch-using layer that follows (pointwise layers on the GEMM path in between use none),
                // reached before anything overwrites the tensor. It goes to the region this layer does not read.
                if (ctx->opt_dual_out && !L.out_int32 && wants_scratch(L, T_o)) {
                    for (int lj = li + 1; lj < n; ++lj) {
                        const qasr_layer& N = tb[lj];
                        const bool gemm_pw = N.kind == QASR_LAYER_PW && !wants_scratch(N, p.t_out[lj]);
                        if (gemm_pw && N.out_buf != L.out_buf) continue;
                        size_t rbytes = 0;
                        char* const home = scratch_region(1 - in_region, rbytes);
                        if (wants_scratch(N, p.t_out[lj]) && N.in_buf == L.out_buf && N.stride == 1 &&
                            N.out_buf != L.out_buf && (size_t)B * L.C_out * T_o <= rbytes)
                            a.yt = (int8_t*)home;
                        break;
                    }
                }
                ctx->yt_written = false;
                rc = run_conv(ctx, a);
                if (a.yt) {
                    // whatever the other region held is gone, whether or not the tensor-core kernel ran
                    ft_buf = ctx->yt_written ? L.out_buf : -1;
                    ft_region = 1 - in_region;
                }
            }
        }
        if (rc) return rc;
        if (!L.out_int32) curC[L.out_buf] = L.C_out;
    }
    ctx->cur_layer = -1;
    memset(&ctx->prefetch, 0, sizeof(ctx->prefetch));
    {
        int rcj = join_side();
        if (rcj) return rcj;
    }
    if (logits && out_scale) {
        QasrLaunchScope ls(ctx, QASR_K_DEQUANT, 0, (double)B * p.C_last * p.T_last * 8);
        QASR_CUDA(ctx, qasr_launch_dequant(logits_q, B, p.C_last, p.T_last, out_scale, logits, ctx->stream));
    }
    return QASR_OK;
}

extern "C" int qasr_encoder_forward(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                                    const int8_t* x, int B, int C_in, int T,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* logits_q, float* logits, const float* out_scale) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x || !logits_q) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_encoder_forward: x or logits_q is NULL");
    if ((logits != nullptr) != (out_scale != nullptr)) QASR_FAIL(ctx, QASR_ERR_NULL, "logits and out_scale must be given together");
    if (!aligned(logits_q, 4) || (logits && (!aligned(logits, 4) || !aligned(out_scale, 4)))) QASR_FAIL(ctx, QASR_ERR_ALIGN, "4-byte alignment required for logits");
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, ctx->err, sizeof(ctx->err));
    if (rc) return rc;
    if (p.total && (!workspace || !aligned(workspace, 256) || workspace_bytes < p.total))
        QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_encoder_forward needs %zu bytes of 256-byte aligned workspace", p.total);
    const char* wlo = (const char*)workspace;
    const char* whi = wlo + p.total;
    auto inside = [&](const void* q) { return p.total && (const char*)q >= wlo && (const char*)q < whi; };
    if (inside(x) || inside(logits_q) || (logits && inside(logits))) QASR_FAIL(ctx, QASR_ERR_ALIAS, "x/logits overlap the workspace");
    if ((const void*)logits_q == (const void*)logits) QASR_FAIL(ctx, QASR_ERR_ALIAS, "logits aliases logits_q");
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));

    // Static-weights option: the regrouped weights in the workspace are those of this very call.
    QasrPlanKey key;
    qasr_plan_key(key, table, n_layers, x, B, C_in, T, workspace, logits_q, logits, out_scale);
    const bool weights_ready = ctx->opt_static_w && ctx->prepared && ctx->prepared_key.same_weights_home(key);
    if (ctx->opt_static_w && !weights_ready) {
        ctx->prepared_key = key;      // this call rebuilds them (stream order makes them ready for the next one)
        ctx->prepared = true;
    }
    if (!ctx->opt_graph || ctx->profiling)
        return enqueue_table(ctx, table, n_layers, p, x, B, (char*)workspace, logits_q, logits, out_scale, weights_ready);

    // Graph path: replay when the call is identical to the cached one, else capture it.
    for (qasr_ctx::GraphEntry& ge : ctx->graphs) {
        if (ge.exec && ge.key == key && ge.regroups == !weights_ready) {
            QASR_CUDA(ctx, cudaGraphLaunch(ge.exec, ctx->stream));
            ctx->launches += ge.nodes;
            ge.last_use = ++ctx->graph_tick;
            return QASR_OK;
        }
    }
    // not cached: the least recently used entry makes room
    qasr_ctx::GraphEntry& slot = ctx->graphs[ctx->graphs[0].last_use <= ctx->graphs[1].last_use ? 0 : 1];
    if (slot.exec) cudaGraphExecDestroy(slot.exec);
    slot = qasr_ctx::GraphEntry();
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    QASR_CUDA(ctx, cudaStreamIsCapturing(ctx->stream, &cs));
    if (cs != cudaStreamCaptureStatusNone)  // the caller is capturing: just enqueue into their graph
        return enqueue_table(ctx, table, n_layers, p, x, B, (char*)workspace, logits_q, logits, out_scale, weights_ready);
    // The legacy default stream cannot be captured, so the capture always runs on a private
    // stream; the instantiated graph is then launched on the caller's stream.
    if (!ctx->capture_stream)
        QASR_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking));
    QASR_CUDA(ctx, cudaStreamBeginCapture(ctx->capture_stream, cudaStreamCaptureModeThreadLocal));
    const int64_t before = ctx->launches;
    cudaStream_t user_stream = ctx->stream;
    ctx->stream = ctx->capture_stream;
    rc = enqueue_table(ctx, table, n_layers, p, x, B, (char*)workspace, logits_q, logits, out_scale, weights_ready, true);
    ctx->stream = user_stream;
    ctx->grid_cap = 0;
    cudaGraph_t g = nullptr;
    cudaError_t ce = cudaStreamEndCapture(ctx->capture_stream, &g);
    const int64_t nodes = ctx->launches - before;
    ctx->launches = before;
    if (rc) {
        if (g) cudaGraphDestroy(g);
        return rc;
    }
    QASR_CUDA(ctx, ce);
    ce = cudaGraphInstantiate(&slot.exec, g, 0);
    cudaGraphDestroy(g);
    if (ce != cudaSuccess) slot.exec = nullptr;
    QASR_CUDA(ctx, ce);
    slot.key = key;
    slot.nodes = nodes;
    slot.regroups = !weights_ready;
    slot.last_use = ++ctx->graph_tick;
    QASR_CUDA(ctx, cudaGraphLaunch(slot.exec, ctx->stream));
    ctx->launches += nodes;
    return QASR_OK;
}

// Streams and events of the pipelined host entry point, created on first use.
static int host_pipeline_init(qasr_ctx* ctx) {
    if (ctx->copy_in) return QASR_OK;
    QASR_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking));
    QASR_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking));
    for (int s = 0; s < 2; ++s) {
        QASR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_in[s], cudaEventDisableTiming));
        QASR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_comp[s], cudaEventDisableTiming));
        QASR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_out[s], cudaEventDisableTiming));
    }
    return QASR_OK;
}

extern "C" int qasr_encoder_host_pipeline_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                                size_t* bytes) {
    if (!bytes) return QASR_ERR_NULL;
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, nullptr, 0);
    if (rc) return rc;
    *bytes = p.total + 2 * staging_for(p, B, C_in, T).total;
    return QASR_OK;
}

extern "C" int qasr_encoder_host_wait(qasr_ctx* ctx, int slot) {
    if (!ctx) return QASR_ERR_NULL;
    if (slot < 0 || slot > 1) QASR_FAIL(ctx, QASR_ERR_SHAPE, "slot %d must be 0 or 1", slot);
    if (!ctx->slot_pending[slot]) return QASR_OK;
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    QASR_CUDA(ctx, cudaEventSynchronize(ctx->ev_out[slot]));
    ctx->slot_pending[slot] = false;
    return QASR_OK;
}

extern "C" int qasr_encoder_forward_host_async(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                                               const int8_t* x_host, int B, int C_in, int T,
                                               void* workspace, size_t workspace_bytes,
                                               int32_t* logits_q_host, float* logits_host, const float* out_scale,
                                               int slot) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x_host || !logits_q_host) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_encoder_forward_host_async: x or logits_q is NULL");
    if (slot < 0 || slot > 1) QASR_FAIL(ctx, QASR_ERR_SHAPE, "slot %d must be 0 or 1", slot);
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, ctx->err, sizeof(ctx->err));
    if (rc) return rc;
    const Staging s = staging_for(p, B, C_in, T);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < p.total + 2 * s.total)
        QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_encoder_forward_host_async needs %zu bytes of 256-byte aligned workspace", p.total + 2 * s.total);
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    QASR_CUDA(ctx, cudaStreamIsCapturing(ctx->stream, &cs));
    if (cs != cudaStreamCaptureStatusNone) QASR_FAIL(ctx, QASR_ERR_CUDA, "qasr_encoder_forward_host_async cannot run inside a stream capture");
    if ((rc = host_pipeline_init(ctx))) return rc;
    // the slot's previous results must have reached the host before its device buffers are written again
    if ((rc = qasr_encoder_host_wait(ctx, slot))) return rc;
    char* st = (char*)workspace + p.total + (size_t)slot * s.total;
    int8_t* x_dev = (int8_t*)(st + s.x);
    int32_t* lq_dev = (int32_t*)(st + s.lq);
    float* lf_dev = logits_host ? (float*)(st + s.lf) : nullptr;
    const size_t n_logit = (size_t)B * p.C_last * p.T_last;
    // input copy on its own stream: it may run while the kernels of the other slot's call still do
    QASR_CUDA(ctx, cudaMemcpyAsync(x_dev, x_host, (size_t)B * C_in * T, cudaMemcpyHostToDevice, ctx->copy_in));
    QASR_CUDA(ctx, cudaEventRecord(ctx->ev_in[slot], ctx->copy_in));
    QASR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_in[slot], 0));
    rc = qasr_encoder_forward(ctx, table, n_layers, x_dev, B, C_in, T, workspace, p.total, lq_dev, lf_dev,
                              lf_dev ? out_scale : nullptr);
    if (rc) return rc;
    QASR_CUDA(ctx, cudaEventRecord(ctx->ev_comp[slot], ctx->stream));
    // The next input copy into this slot cannot overtake these kernels: the call that issues it first waits, on
    // the host, for this call's results (above). No device-side wait is put into the copy stream for it: stream
    // order would make the OTHER slot's next input copy wait for these kernels as well, and that copy is the one
    // that has to run beside them.
    // result copies on a third stream: they overlap the next call's kernels
    QASR_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_out, ctx->ev_comp[slot], 0));
    QASR_CUDA(ctx, cudaMemcpyAsync(logits_q_host, lq_dev, n_logit * 4, cudaMemcpyDeviceToHost, ctx->copy_out));
    if (lf_dev) QASR_CUDA(ctx, cudaMemcpyAsync(logits_host, lf_dev, n_logit * 4, cudaMemcpyDeviceToHost, ctx->copy_out));
    QASR_CUDA(ctx, cudaEventRecord(ctx->ev_out[slot], ctx->copy_out));
    ctx->slot_pending[slot] = true;
    return QASR_OK;
}

extern "C" int qasr_encoder_forward_host(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                                         const int8_t* x_host, int B, int C_in, int T,
                                         void* workspace, size_t workspace_bytes,
                                         int32_t* logits_q_host, float* logits_host, const float* out_scale) {
    if (!ctx) return QASR_ERR_NULL;
    if (!x_host || !logits_q_host) QASR_FAIL(ctx, QASR_ERR_NULL, "qasr_encoder_forward_host: x or logits_q is NULL");
    TablePlan p;
    int rc = plan_table(table, n_layers, B, C_in, T, p, ctx->err, sizeof(ctx->err));
    if (rc) return rc;
    const Staging s = staging_for(p, B, C_in, T);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < p.total + s.total)
        QASR_FAIL(ctx, QASR_ERR_WORKSPACE, "qasr_encoder_forward_host needs %zu bytes of 256-byte aligned workspace", p.total + s.total);
    char* st = (char*)workspace + p.total;
    int8_t* x_dev = (int8_t*)(st + s.x);
    int32_t* lq_dev = (int32_t*)(st + s.lq);
    float* lf_dev = logits_host ? (float*)(st + s.lf) : nullptr;
    const size_t n_logit = (size_t)B * p.C_last * p.T_last;
    QASR_CUDA(ctx, cudaSetDevice(ctx->device));
    QASR_CUDA(ctx, cudaMemcpyAsync(x_dev, x_host, (size_t)B * C_in * T, cudaMemcpyHostToDevice, ctx->stream));
    rc = qasr_encoder_forward(ctx, table, n_layers, x_dev, B, C_in, T, workspace, p.total, lq_dev, lf_dev,
                              lf_dev ? out_scale : nullptr);
    if (rc) return rc;
    QASR_CUDA(ctx, cudaMemcpyAsync(logits_q_host, lq_dev, n_logit * 4, cudaMemcpyDeviceToHost, ctx->stream));
    if (lf_dev) QASR_CUDA(ctx, cudaMemcpyAsync(logits_host, lf_dev, n_logit * 4, cudaMemcpyDeviceToHost, ctx->stream));
    QASR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return QASR_OK;
}
