// Generic kernels: correct for any shape and alignment.  They are the path for shapes the
// tensor-core and vectorised kernels do not take (odd sizes, stride/dilation 2, tiny channel
// counts) and for the element-wise steps (residual add, final dequantisation).
#include <cstring>

#include "qasr_device.cuh"
#include "sm100_ptx.cuh"

namespace qasr {

// ------------------------------------------------------------------------------------------
// Depthwise K-tap convolution + requant, one (b, c) row segment per block.
// ------------------------------------------------------------------------------------------
constexpr int DWG_THREADS = 128;
constexpr int DWG_TILE = 512;                                  // outputs per block
constexpr int DWG_SPAN_MAX = (DWG_TILE - 1) * 2 + 126 * 2 + 1;  // stride <= 2, (K-1)*dilation <= 252

__global__ void __launch_bounds__(DWG_THREADS)
dw_conv_generic_kernel(QasrDwArgs a, unsigned* status) {
    __shared__ int8_t xs[DWG_SPAN_MAX + 3];
    __shared__ int8_t ws[128];
    const int c = blockIdx.y, b = blockIdx.z;
    const int t0 = blockIdx.x * DWG_TILE;
    const int pad = a.dilation * (a.K - 1) / 2;
    const int n_out = min(DWG_TILE, a.T_out - t0);
    const int span = (n_out - 1) * a.stride + (a.K - 1) * a.dilation + 1;
    const int8_t* xr = a.x + ((size_t)b * a.C + c) * a.T;
    const int g0 = t0 * a.stride - pad;
    for (int p = threadIdx.x; p < span; p += DWG_THREADS) {
        const int g = g0 + p;
        xs[p] = (g >= 0 && g < a.T) ? xr[g] : (int8_t)0;
    }
    for (int k = threadIdx.x; k < a.K; k += DWG_THREADS) ws[k] = a.w[(size_t)c * a.K + k];
    int m, s;
    load_rq(a.mult, a.shift, c, m, s, status);
    __syncthreads();
    int8_t* yr = a.y + ((size_t)b * a.C + c) * a.T_out + t0;
    for (int j = threadIdx.x; j < n_out; j += DWG_THREADS) {
        int acc = 0;
        const int base = j * a.stride;
        for (int k = 0; k < a.K; ++k) acc += (int)ws[k] * (int)xs[base + k * a.dilation];
        yr[j] = (int8_t)requant64(acc, m, s);
    }
}

// ------------------------------------------------------------------------------------------
// Pointwise / dense K-tap convolution with the fused epilogue.
// Block tile: 64 output channels x 64 output frames of one utterance; 256 threads, 4x4 each.
// ------------------------------------------------------------------------------------------
constexpr int CG_THREADS = 256;
constexpr int CG_TO = 64;    // output channels per block
constexpr int CG_TT = 64;    // output frames per block
constexpr int CG_IC = 32;    // input channels per smem chunk
constexpr int CG_XS = (CG_TT - 1) * 2 + 126 * 2 + 1;  // 379
constexpr int CG_XS_PITCH = 384;
static_assert(CG_XS <= CG_XS_PITCH, "input tile must hold the widest receptive field");

__global__ void __launch_bounds__(CG_THREADS)
conv_generic_kernel(QasrConvArgs a, unsigned* status) {
    __shared__ int8_t xs[CG_IC][CG_XS_PITCH];
    __shared__ int8_t ws[CG_TO][CG_IC + 4];
    const int b = blockIdx.z;
    const int o0 = blockIdx.y * CG_TO;
    const int t0 = blockIdx.x * CG_TT;
    const int pad = a.dilation * (a.K - 1) / 2;
    const int span = (CG_TT - 1) * a.stride + (a.K - 1) * a.dilation + 1;
    const int g0 = t0 * a.stride - pad;
    const int tx = threadIdx.x % 16;   // frames tx, tx+16, tx+32, tx+48
    const int ty = threadIdx.x / 16;   // channels ty*4 .. ty*4+3

    int acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

    for (int ic0 = 0; ic0 < a.C_in; ic0 += CG_IC) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < CG_IC * span; idx += CG_THREADS) {
            const int i = idx / span, p = idx - i * span;
            const int g = g0 + p;
            int8_t v = 0;
            if (ic0 + i < a.C_in && g >= 0 && g < a.T)
                v = a.x[((size_t)b * a.C_in + ic0 + i) * a.T + g];
            xs[i][p] = v;
        }
        for (int k = 0; k < a.K; ++k) {
            __syncthreads();
            for (int idx = threadIdx.x; idx < CG_TO * CG_IC; idx += CG_THREADS) {
                const int oo = idx / CG_IC, ii = idx - oo * CG_IC;
                int8_t v = 0;
                if (o0 + oo < a.C_out && ic0 + ii < a.C_in)
                    v = a.w[((size_t)(o0 + oo) * a.C_in + ic0 + ii) * a.K + k];
                ws[oo][ii] = v;
            }
            __syncthreads();
            const int xoff = k * a.dilation;
#pragma unroll 4
            for (int ii = 0; ii < CG_IC; ++ii) {
                int wv[4], xv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) wv[i] = ws[ty * 4 + i][ii];
#pragma unroll
                for (int j = 0; j < 4; ++j) xv[j] = xs[ii][(tx + 16 * j) * a.stride + xoff];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] += wv[i] * xv[j];
            }
        }
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int o = o0 + ty * 4 + i;
        if (o >= a.C_out) continue;
        const int bias = a.bias ? a.bias[o] : 0;
        int m = 0, s = 1;
        if (!a.y_int32) load_rq(a.mult, a.shift, o, m, s, status);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = t0 + tx + 16 * j;
            if (t >= a.T_out) continue;
            const size_t idx = ((size_t)b * a.C_out + o) * a.T_out + t;
            const int v = acc[i][j] + bias;
            if (a.y_int32) {
                a.y_int32[idx] = v;
            } else {
                int q = requant64(v, m, s);
                if (a.terms.n > 0) q = residual_stage(q, a.terms, idx, a.relu);
                else if (a.relu) q = max(q, 0);
                a.y[idx] = (int8_t)q;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Integer residual add, element-wise.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
residual_add_kernel(QasrTerms t, size_t n, int relu, int8_t* y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        long long v = 0;
        for (int j = 0; j < t.n; ++j) v += rescale_term((int)t.ptr[j][i], t.mult[j], t.shift[j]);
        if (relu && v < 0) v = 0;
        y[i] = (int8_t)clamp_i8_ll(v);
    }
}

// 16 elements per thread; requires every pointer 16-byte aligned and n % 16 == 0.
__global__ void __launch_bounds__(256)
residual_add_vec_kernel(QasrTerms t, size_t n_vec, int relu, int8_t* y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        long long v[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = 0;
        for (int j = 0; j < t.n; ++j) {
            const int4 q = __ldg(reinterpret_cast<const int4*>(t.ptr[j]) + i);
            const int words[4] = {q.x, q.y, q.z, q.w};
            const int m = t.mult[j], s = t.shift[j];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int qv = (int)(int8_t)((words[e >> 2] >> ((e & 3) * 8)) & 0xff);
                v[e] += rescale_term(qv, m, s);
            }
        }
        int out[4] = {0, 0, 0, 0};
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            long long r = v[e];
            if (relu && r < 0) r = 0;
            out[e >> 2] |= ((int)clamp_i8_ll(r) & 0xff) << ((e & 3) * 8);
        }
        reinterpret_cast<int4*>(y)[i] = make_int4(out[0], out[1], out[2], out[3]);
    }
}

// ------------------------------------------------------------------------------------------
// Final dequantisation: one fp32 multiply per logit.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
dequant_kernel(const int32_t* acc, int C, int T, size_t n, const float* scale, float* out) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const int c = (int)((i / (size_t)T) % (size_t)C);
        out[i] = __fmul_rn(__int2float_rn(acc[i]), scale[c]);
    }
}

// ------------------------------------------------------------------------------------------
// Integer GLU: the input holds 2C channels, a = channels [0, C), gate = channels [C, 2C).
//   u = min(|g|, q_c); p = q_c - u; h = 2 q_c^2 - p^2; sig = g >= 0 ? h : 2 q_c^2 - h
//   y = sat8(RS(a * sig * mult[c], shift[c]))
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
glu_kernel(const int8_t* x, int C, int T, size_t n, int q_c, const int32_t* mult, const uint8_t* shift,
           int8_t* y, unsigned* status) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const int t = (int)(i % (size_t)T);
        const size_t bc = i / (size_t)T;
        const int c = (int)(bc % (size_t)C);
        const size_t b = bc / (size_t)C;
        int m, s;
        load_rq(mult, shift, c, m, s, status);
        const size_t ia = (b * 2 * C + c) * (size_t)T + t;
        const int a = x[ia];
        const int g = x[ia + (size_t)C * T];
        const int u = min(abs(g), q_c);
        const int pq = q_c - u;
        const int full = 2 * q_c * q_c;
        const int h = full - pq * pq;
        const int sig = g >= 0 ? h : full - h;
        const long long prod = (long long)(a * sig) * (long long)m + (1LL << (s - 1));
        y[i] = (int8_t)clamp_i8_ll(prod >> s);
    }
}

// The same gate, 16 consecutive frames of one channel per thread (16-byte loads and stores); T16 = T / 16.
// The channel's dyadic constant is normalised to a shift of at least 32 where the multiplier has the head-room
// ((m << k, s + k) is the same number), so that the rescaling is the high word of one multiply-add.
template <int W>
__device__ __forceinline__ void glu_word(uint32_t aw, uint32_t gw, int q_c, int full, int mn, long long half, int sn,
                                         bool fast, int (&q)[16]) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int a = e == 0 ? ptx::sext_byte<0>(aw) : e == 1 ? ptx::sext_byte<1>(aw) : e == 2 ? ptx::sext_byte<2>(aw) : ptx::sext_byte<3>(aw);
        const int g = e == 0 ? ptx::sext_byte<0>(gw) : e == 1 ? ptx::sext_byte<1>(gw) : e == 2 ? ptx::sext_byte<2>(gw) : ptx::sext_byte<3>(gw);
        const int pq = q_c - min(abs(g), q_c);
        const int h = full - pq * pq;
        const int sig = g >= 0 ? h : full - h;
        const int v = a * sig;                          // |v| <= 128 * 2 * 128^2 < 2^23
        q[4 * W + e] = fast ? ptx::mad_hi64(v, mn, half) >> (sn - 32)
                            : (int)clamp_i8_ll(((long long)v * (long long)mn + half) >> sn);
    }
}

__global__ void __launch_bounds__(256)
glu_vec16_kernel(const int8_t* __restrict__ x, int C, int T16, unsigned items, int q_c, const int32_t* mult,
                 const uint8_t* shift, int8_t* __restrict__ y, unsigned* status) {
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    // launched with programmatic early launch inside a layer table: the channel's constants are fetched while
    // the kernel that writes x still runs; x is read behind the dependency wait
    ptx::grid_dep_launch();
    if (i >= items) return;
    const unsigned t16 = i % (unsigned)T16, bc = i / (unsigned)T16;
    const unsigned c = bc % (unsigned)C, b = bc / (unsigned)C;
    const size_t row = (size_t)T16 * 16;
    const size_t ia = ((size_t)b * 2 * C + c) * row + (size_t)t16 * 16;
    int m, s;
    load_rq(mult, shift, (int)c, m, s, status);
    ptx::grid_dep_wait();
    const int4 av = __ldg(reinterpret_cast<const int4*>(x + ia));
    const int4 gv = __ldg(reinterpret_cast<const int4*>(x + ia + (size_t)C * row));
    const int kmax = min(__clz(m) - 1, 62 - s);
    const int k = (s <= 32 && 32 - s <= kmax) ? 32 - s : max(kmax, 0);
    const int mn = m << k, sn = s + k;
    const long long half = 1LL << (sn - 1);
    const bool fast = sn >= 32;
    const int full = 2 * q_c * q_c;
    int q[16];
    glu_word<0>((uint32_t)av.x, (uint32_t)gv.x, q_c, full, mn, half, sn, fast, q);
    glu_word<1>((uint32_t)av.y, (uint32_t)gv.y, q_c, full, mn, half, sn, fast, q);
    glu_word<2>((uint32_t)av.z, (uint32_t)gv.z, q_c, full, mn, half, sn, fast, q);
    glu_word<3>((uint32_t)av.w, (uint32_t)gv.w, q_c, full, mn, half, sn, fast, q);
    int4 out;
    out.x = (int)ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
    out.y = (int)ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
    out.z = (int)ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
    out.w = (int)ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
    *reinterpret_cast<int4*>(y + ((size_t)bc * row + (size_t)t16 * 16)) = out;
}

}  // namespace qasr

cudaError_t qasr_launch_glu(const int8_t* x, int B, int C, int T, int q_c, const int32_t* mult,
                            const uint8_t* shift, int8_t* y, unsigned* status, cudaStream_t st, int early_launch) {
    const size_t n = (size_t)B * C * T;
    if (T % 16 == 0 && (((uintptr_t)x | (uintptr_t)y) & 15u) == 0 && n / 16 < 0x7fffffffu) {
        const unsigned items = (unsigned)(n / 16);
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((items + 255) / 256); cfg.blockDim = dim3(256); cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = early_launch ? 1 : 0;
        cfg.attrs = attr; cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, qasr::glu_vec16_kernel, x, C, T / 16, items, q_c, mult, shift, y, status);
    }
    const unsigned blocks = (unsigned)((n + 255) / 256 < 148u * 16u ? (n + 255) / 256 : 148u * 16u);
    qasr::glu_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(x, C, T, n, q_c, mult, shift, y, status);
    return cudaGetLastError();
}

cudaError_t qasr_launch_dw_generic(const QasrDwArgs& a, unsigned* status, cudaStream_t st) {
    dim3 grid((a.T_out + qasr::DWG_TILE - 1) / qasr::DWG_TILE, a.C, a.B);
    qasr::dw_conv_generic_kernel<<<grid, qasr::DWG_THREADS, 0, st>>>(a, status);
    return cudaGetLastError();
}

cudaError_t qasr_launch_conv_generic(const QasrConvArgs& a, unsigned* status, cudaStream_t st) {
    dim3 grid((a.T_out + qasr::CG_TT - 1) / qasr::CG_TT, (a.C_out + qasr::CG_TO - 1) / qasr::CG_TO, a.B);
    qasr::conv_generic_kernel<<<grid, qasr::CG_THREADS, 0, st>>>(a, status);
    return cudaGetLastError();
}

cudaError_t qasr_launch_residual_add(const QasrTerms& t, size_t n, int relu, int8_t* y,
                                     unsigned* status, cudaStream_t st) {
    (void)status;
    bool vec = (n % 16 == 0) && ((uintptr_t)y % 16 == 0);
    for (int j = 0; j < t.n; ++j) vec = vec && ((uintptr_t)t.ptr[j] % 16 == 0);
    if (vec) {
        const size_t nv = n / 16;
        const unsigned blocks = (unsigned)((nv + 255) / 256 < 148u * 16u ? (nv + 255) / 256 : 148u * 16u);
        qasr::residual_add_vec_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(t, nv, relu, y);
    } else {
        const unsigned blocks = (unsigned)((n + 255) / 256 < 148u * 16u ? (n + 255) / 256 : 148u * 16u);
        qasr::residual_add_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(t, n, relu, y);
    }
    return cudaGetLastError();
}

cudaError_t qasr_launch_dequant(const int32_t* acc, int B, int C, int T, const float* scale,
                                float* out, cudaStream_t st) {
    const size_t n = (size_t)B * C * T;
    const unsigned blocks = (unsigned)((n + 255) / 256 < 148u * 8u ? (n + 255) / 256 : 148u * 8u);
    qasr::dequant_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(acc, C, T, n, scale, out);
    return cudaGetLastError();
}
