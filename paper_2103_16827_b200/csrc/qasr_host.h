// Host-side context and fast-path hooks (internal).
#pragma once

#include <cstring>
#include <utility>
#include <vector>

#include "qasr_internal.h"

struct QasrPlanKey {
    std::vector<char> table;   // byte copy of the layer table
    const void* ptrs[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    int B = 0, C_in = 0, T = 0;
    bool operator==(const QasrPlanKey& o) const {
        return B == o.B && C_in == o.C_in && T == o.T && table == o.table &&
               std::memcmp(ptrs, o.ptrs, sizeof(ptrs)) == 0;
    }
    // Same layer table, shape and workspace (whatever the input and output tensors are): the regrouped
    // weights that one such call left in the workspace are the ones the other needs.
    bool same_weights_home(const QasrPlanKey& o) const {
        return B == o.B && C_in == o.C_in && T == o.T && ptrs[1] == o.ptrs[1] && table == o.table;
    }
};

// kernel ids reported by the profiler
enum QasrKernelId {
    QASR_K_DW_GENERIC = 1, QASR_K_CONV_GENERIC = 2, QASR_K_RESIDUAL_ADD = 3, QASR_K_DEQUANT = 4,
    QASR_K_DW_DP4A = 5, QASR_K_GEMM_TC = 6, QASR_K_CONV_TC = 8, QASR_K_GLU = 9,
    QASR_K_DW_TC = 10, QASR_K_CONV_PREP = 11
};

struct QasrProfRec {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int layer = -1, kernel = 0;
    double macs = 0, bytes = 0;
};

struct qasr_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    unsigned* d_status = nullptr;
    int sm_count = 148;
    int cc_major = 0;
    bool opt_graph = true, opt_tc = true, opt_pdl = true, opt_static_w = false;
    int force_gemm_bn = 0, force_dw_nt = 0;      // tuning aids: 0 = automatic
    // Side branch of a captured layer table: a convolution whose result is needed only several layers later
    // (a block's residual projection) runs on a second stream, on the SMs the main chain leaves idle.
    bool opt_side = true;
    // A K-tap convolution on the tensor cores writes its output a second time, frame-major, where the next
    // K-tap convolution of the table reads it (that one then needs no transpose kernel).
    bool opt_dual_out = true;
    // Set around a launch whose CTAs must not become resident before the previous kernel has ended: while a side
    // branch is pending, early CTAs of a long main-chain kernel would sit in their dependency wait on the very SMs
    // the branch's next kernel needs.
    bool hold_early_launch = false;
    bool yt_written = false;                     // set by the launch that wrote QasrConvArgs::yt
    int grid_cap = 0;                            // > 0: persistent kernels launch at most this many CTAs
    cudaStream_t side_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_side = nullptr;
    int64_t launches = 0;
    char err[512] = {0};
    // cached CUDA graphs of the last qasr_encoder_forward calls (two entries, least recently used one is
    // replaced: a caller that alternates between two sets of buffers replays both)
    struct GraphEntry {
        cudaGraphExec_t exec = nullptr;
        QasrPlanKey key;
        int64_t nodes = 0;
        bool regroups = true;        // the graph contains the weight regrouping kernels
        uint64_t last_use = 0;
    };
    GraphEntry graphs[2];
    uint64_t graph_tick = 0;
    cudaStream_t capture_stream = nullptr;
    // pipelined host entry point: copy streams and per-slot events (created on first use)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_comp[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    bool slot_pending[2] = {false, false};
    // static-weights option: the call whose regrouped weights the workspace currently holds
    QasrPlanKey prepared_key;
    bool prepared = false;
    // profile mode
    bool profiling = false;
    int cur_layer = -1;
    std::vector<QasrProfRec> prof;
    // driver entry point for tensor-map encoding (resolved once)
    void* encode_tiled = nullptr;
    // constants of the kernel that the layer table launches next (consumed and cleared by the next launch)
    QasrPrefetch prefetch = {};
    // scratch lent by the caller for single qasr_conv calls (qasr_set_conv_scratch)
    void* conv_scratch = nullptr;
    size_t conv_scratch_bytes = 0;
};

inline void qasr_plan_key(QasrPlanKey& k, const qasr_layer* table, int n, const void* x, int B, int C_in,
                          int T, const void* ws, const void* lq, const void* lf, const void* sc) {
    k.table.assign((const char*)table, (const char*)table + sizeof(qasr_layer) * (size_t)n);
    k.ptrs[0] = x; k.ptrs[1] = ws; k.ptrs[2] = lq; k.ptrs[3] = lf; k.ptrs[4] = sc;
    k.B = B; k.C_in = C_in; k.T = T;
}

inline void qasr_plan_cache_clear(qasr_ctx* ctx) {
    for (qasr_ctx::GraphEntry& g : ctx->graphs) {
        if (g.exec) cudaGraphExecDestroy(g.exec);
        g = qasr_ctx::GraphEntry();
    }
}

// Brackets one kernel launch with events when the context is in profile mode, and counts it.
struct QasrLaunchScope {
    qasr_ctx* ctx;
    QasrProfRec rec;
    QasrLaunchScope(qasr_ctx* c, int kernel, double macs, double bytes) : ctx(c) {
        ctx->launches++;
        if (!ctx->profiling) return;
        rec.layer = ctx->cur_layer; rec.kernel = kernel; rec.macs = macs; rec.bytes = bytes;
        if (cudaEventCreate(&rec.e0) != cudaSuccess || cudaEventCreate(&rec.e1) != cudaSuccess) { rec.e0 = rec.e1 = nullptr; return; }
        cudaEventRecord(rec.e0, ctx->stream);
    }
    ~QasrLaunchScope() {
        if (!ctx->profiling || !rec.e0) return;
        cudaEventRecord(rec.e1, ctx->stream);
        ctx->prof.push_back(rec);
    }
};

inline double qasr_dw_macs(const QasrDwArgs& a) { return (double)a.B * a.C * a.T_out * a.K; }
inline double qasr_dw_bytes(const QasrDwArgs& a) { return (double)a.B * a.C * ((double)a.T + a.T_out) + (double)a.C * a.K; }
inline double qasr_conv_macs(const QasrConvArgs& a) { return (double)a.B * a.C_out * a.T_out * a.C_in * a.K; }
inline double qasr_conv_bytes(const QasrConvArgs& a) {
    const double out = (double)a.B * a.C_out * a.T_out;
    return (double)a.B * a.C_in * a.T + out * (a.y_int32 ? 4 : 1) + (a.terms.n > 1 ? (a.terms.n - 1) * out : 0) +
           (double)a.C_out * a.C_in * a.K + 9.0 * a.C_out;
}

// True if the residual stage of an epilogue can be carried in 32-bit arithmetic without changing a bit:
// every product q * mult + 2^(shift-1) with |q| <= 128 fits int32 (mult < 2^23, shift <= 30), and so does
// the sum of the rescaled terms, each of which is at most ((128 * mult) >> shift) + 1 in magnitude.
inline bool qasr_terms_fit_int32(const QasrTerms& t) {
    long long sum = 0;
    for (int j = 0; j < t.n; ++j) {
        if (t.mult[j] < 0 || t.mult[j] >= (1 << 23) || t.shift[j] < 1 || t.shift[j] > 30) return false;
        sum += ((128LL * t.mult[j]) >> t.shift[j]) + 1;
    }
    return sum < (1LL << 31);
}

// CTAs a one-CTA-per-SM persistent kernel may launch: every SM, unless a side branch shares the GPU.
inline int qasr_grid_slots(const qasr_ctx* ctx) {
    return ctx->grid_cap > 0 && ctx->grid_cap < ctx->sm_count ? ctx->grid_cap : ctx->sm_count;
}

// Launches a kernel whose prologue may overlap the tail of the previous kernel in the stream
// (programmatic dependent launch); the kernel itself must execute griddepcontrol.wait before it
// touches anything an earlier kernel wrote or still reads.
template <typename... KArgs, typename... Args>
inline cudaError_t qasr_launch_overlapped(qasr_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                          Args&&... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = ctx->opt_pdl && !ctx->hold_early_launch ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// One-time host set-up of the fast paths (driver entry points, kernel attributes).
int qasr_host_init(qasr_ctx* ctx);

// Fast paths. Each returns 1 if it enqueued the operation, 0 if the shape/alignment is not one it
// takes (the caller then uses the generic kernel), or a negative QASR_ERR_* code.
int qasr_try_dw_fast(qasr_ctx* ctx, const QasrDwArgs& a);
int qasr_try_conv_tc(qasr_ctx* ctx, const QasrConvArgs& a);
// Scratch bytes the tensor-core path of a K-tap convolution wants in QasrConvArgs::scratch.
size_t qasr_conv_tc_scratch_bytes(int B, int C_in, int C_out, int T, int K, int stride);
// The two parts of it: the frame-major input copy and the regrouped weights.
size_t qasr_conv_tc_input_bytes(int B, int C_in, int T, int stride);
size_t qasr_conv_tc_weight_bytes(int C_in, int C_out, int K);
// True if the pointwise GEMM kernel takes this shape (then no scratch is needed).
bool qasr_conv_shape_fits_gemm(int C_in, int K, int stride, int dilation, int T_out);
