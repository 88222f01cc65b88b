// qasr_tcs_block_noalloc: the time-channel-separable block for callers that must not allocate.
//
// qasr_tcs_block keeps the depthwise output in a caller-supplied workspace and needs a context,
// whose creation calls cudaMalloc.  Some callers can do neither: a streaming recogniser's audio
// callback that runs under a fixed device-memory budget, an inference-server plugin whose enqueue
// hook is forbidden to touch the allocator, a process in which another component has reserved all
// device memory up front.  For them the depthwise output lives in the static device array below,
// which is part of the library image: every GPU that loads the library holds
// QASR_NOALLOC_SCRATCH_BYTES (plus a status word) until the process exits, and nothing is ever
// allocated or freed by this entry point.
//
// The array's name is only a host-side handle; the device address is obtained once per device with
// cudaGetSymbolAddress (that device current) and handed to the kernels.
#include <mutex>

#include "qasr_host.h"

int qasr_gemm_tc_init(qasr_ctx* ctx);
int qasr_dw_tc_init(qasr_ctx* ctx);

namespace {

static __device__ __align__(256) unsigned char g_noalloc_scratch[QASR_NOALLOC_SCRATCH_BYTES];
static __device__ __align__(256) unsigned int g_noalloc_status[64];

constexpr int kMaxDevices = 64;

struct DeviceSetup {
    bool ready = false;
    void* scratch = nullptr;
    unsigned* status = nullptr;
    int sm_count = 0;
    int cc_major = 0;
    void* encode_tiled = nullptr;
    bool tc_ok = false;
};

std::mutex g_mutex;
DeviceSetup g_dev[kMaxDevices];

// Once per device, with that device current.
int setup_device(int device, DeviceSetup** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSetup& d = g_dev[device];
    if (!d.ready) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return QASR_ERR_CUDA;
        }
        void* s = nullptr;
        if (cudaGetSymbolAddress(&s, g_noalloc_status) != cudaSuccess || !s) {
            cudaGetLastError();
            return QASR_ERR_CUDA;
        }
        d.scratch = p;
        d.status = (unsigned*)s;
        if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
            cudaGetLastError();
            return QASR_ERR_CUDA;
        }
        if (d.cc_major == 10) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
                qres == cudaDriverEntryPointSuccess && fn) {
                qasr_ctx probe;
                probe.device = device;
                if (qasr_gemm_tc_init(&probe) == QASR_OK && qasr_dw_tc_init(&probe) == QASR_OK) {
                    d.encode_tiled = fn;
                    d.tc_ok = true;
                }
            }
            cudaGetLastError();
        }
        d.ready = true;
    }
    *out = &d;
    return QASR_OK;
}

inline bool aligned4(const void* p) { return ((uintptr_t)p & 3u) == 0; }

}  // namespace

extern "C" int qasr_tcs_block_noalloc(int device, void* cuda_stream,
                                      const int8_t* x, int B, int C_in, int T,
                                      const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                                      const int8_t* w_pw, int C_out, const int32_t* bias, int32_t max_abs_bias,
                                      qasr_requant rq_pw, int relu, int8_t* y, int wait) {
    // ---- host-side validation: nothing is launched on error
    if (!x || !w_dw || !w_pw || !y || !rq_dw.mult || !rq_dw.shift || !rq_pw.mult || !rq_pw.shift) return QASR_ERR_NULL;
    if (device < 0 || device >= kMaxDevices) return QASR_ERR_SHAPE;
    if (B <= 0 || B > 65535 || C_in <= 0 || C_in > 65535 || C_out <= 0 || T <= 0) return QASR_ERR_SHAPE;
    if (K < 1 || K > 127 || (K % 2) == 0 || (stride != 1 && stride != 2) || (dilation != 1 && dilation != 2))
        return QASR_ERR_SHAPE;
    if (!aligned4(rq_dw.mult) || !aligned4(rq_pw.mult) || (bias && !aligned4(bias))) return QASR_ERR_ALIGN;
    if (max_abs_bias < 0) return QASR_ERR_SHAPE;
    if ((long long)K * 127 * 128 >= (1LL << 31)) return QASR_ERR_OVERFLOW_RISK;
    if ((long long)C_in * 127 * 128 + (bias ? (long long)max_abs_bias : 0) >= (1LL << 31)) return QASR_ERR_OVERFLOW_RISK;
    if ((const void*)x == (const void*)y) return QASR_ERR_ALIAS;
    const int T_out = (T - 1) / stride + 1;
    const unsigned long long need = (unsigned long long)B * C_in * T_out;   // the depthwise output
    if (need > QASR_NOALLOC_SCRATCH_BYTES) return QASR_ERR_TOO_LARGE;
    if ((unsigned long long)B * C_out * T_out >= (1ull << 40)) return QASR_ERR_SHAPE;

    if (cudaSetDevice(device) != cudaSuccess) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    DeviceSetup* d = nullptr;
    int rc = setup_device(device, &d);
    if (rc != QASR_OK) return rc;

    // A context on the stack stands in for qasr_create's: same launch helpers, static status word.
    qasr_ctx ctx;
    ctx.device = device;
    ctx.stream = (cudaStream_t)cuda_stream;
    ctx.d_status = d->status;
    ctx.sm_count = d->sm_count;
    ctx.cc_major = d->cc_major;
    ctx.encode_tiled = d->encode_tiled;
    ctx.opt_tc = d->tc_ok;
    ctx.opt_graph = false;

    int8_t* h = (int8_t*)d->scratch;
    QasrDwArgs dw{x, w_dw, rq_dw.mult, rq_dw.shift, h, B, C_in, T, T_out, K, stride, dilation};
    QasrConvArgs pw;
    memset(&pw, 0, sizeof(pw));
    pw.x = h; pw.w = w_pw; pw.bias = bias; pw.mult = rq_pw.mult; pw.shift = rq_pw.shift; pw.y = y;
    pw.B = B; pw.C_in = C_in; pw.C_out = C_out; pw.T = T_out; pw.T_out = T_out;
    pw.K = 1; pw.stride = 1; pw.dilation = 1; pw.relu = relu ? 1 : 0;

    int used = qasr_try_dw_fast(&ctx, dw);
    if (used < 0) return used;
    if (!used && qasr_launch_dw_generic(dw, ctx.d_status, ctx.stream) != cudaSuccess) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    used = qasr_try_conv_tc(&ctx, pw);
    if (used < 0) return used;
    if (!used && qasr_launch_conv_generic(pw, ctx.d_status, ctx.stream) != cudaSuccess) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    if (!wait) return QASR_OK;

    unsigned st = 0;
    if (cudaStreamSynchronize(ctx.stream) != cudaSuccess ||
        cudaMemcpy(&st, d->status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    if (st) {
        if (cudaMemset(d->status, 0, sizeof(st)) != cudaSuccess) cudaGetLastError();
        if (st & QASR_STATUS_TIMEOUT) return QASR_ERR_DEVICE_TIMEOUT;
        if (st & QASR_STATUS_RANGE) return QASR_ERR_RANGE;
    }
    return QASR_OK;
}
