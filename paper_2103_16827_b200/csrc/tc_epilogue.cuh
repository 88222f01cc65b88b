// Epilogue arithmetic shared by the tensor-core convolution kernels: per-channel requantisation
// constants in a normalised form, the 16-column requantiser, and the full epilogue with residual terms
// (bias -> requant -> clamp -> rescaled residual terms -> ReLU -> clamp).
#pragma once

#include "qasr_device.cuh"
#include "sm100_ptx.cuh"

namespace qasr {
namespace tc {

// Per-channel requantisation constants, normalised so that the shift is >= 32 whenever the
// multiplier has enough head-room: (m << k, s + k) encodes the same dyadic number exactly.
struct ChannelRq {
    int m, s;          // normalised multiplier and shift
    long long c64;     // bias * m + 2^(s-1): the rounding constant with the bias folded in
    int fast;          // s >= 32: result = hi32(acc * m + c64) >> (s - 32)
};

__device__ __forceinline__ ChannelRq make_rq(int bias, int m, int s) {
    ChannelRq r;
    const int kmax = min(__clz(m) - 1, 62 - s);
    const int k = (s <= 32 && 32 - s <= kmax) ? 32 - s : kmax;   // land on shift 32 when possible
    r.m = m << k;
    r.s = s + k;
    r.c64 = (long long)bias * (long long)r.m + (1LL << (r.s - 1));
    r.fast = r.s >= 32;
    return r;
}

__device__ __forceinline__ int requant_fast(int acc, int m, long long c64, int sh) {
    const long long p = (long long)acc * (long long)m + c64;
    return (int)(p >> 32) >> sh;             // not yet clamped; |value| < 2^31
}

__device__ __forceinline__ int requant_slow(int acc, const ChannelRq& r) {
    const long long p = (long long)acc * (long long)r.m + r.c64;
    const long long v = p >> r.s;
    return (int)(v > 127 ? 127 : (v < -128 ? -128 : v));
}

// The common epilogue (no residual terms): 16 accumulators -> 16 int8. MODE 0: every lane's shift is
// exactly 32, the result is the high word of acc * m + c64; MODE 1: shift >= 32, one more shift.
template <int MODE, bool RELU>
__device__ __forceinline__ int4 requant16(const uint32_t (&r)[16], const ChannelRq& rq) {
    int q[16];
    const int sh = rq.s - 32;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        int v = ptx::mad_hi64((int)r[i], rq.m, rq.c64);
        if (MODE == 1) v >>= sh;
        q[i] = v;
    }
    // saturate to int8 first, then ReLU on the packed bytes: max(sat8(v), 0) = sat8(max(v, 0))
    uint4 out;
    out.x = ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
    out.y = ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
    out.z = ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
    out.w = ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
    if (RELU) {
        out.x = ptx::relu4_s8(out.x); out.y = ptx::relu4_s8(out.y);
        out.z = ptx::relu4_s8(out.z); out.w = ptx::relu4_s8(out.w);
    }
    return make_int4((int)out.x, (int)out.y, (int)out.z, (int)out.w);
}

// The epilogue of a block's last layer in its common form: one residual tensor beside the layer's own output, every
// constant small enough for 32-bit products (the caller has checked both, and that every lane's shift is >= 32).
// `res` holds the residual's 16 int8 of this thread's channel, fetched a chunk ahead by the caller.
//   a = sat8(RS((acc + bias) * m, s));  v = RS(a * m0, s0) + RS(r * m1, s1);  y = sat8(relu?(v))
struct ResidualOne {
    int m0, s0, h0;    // the layer's own output: multiplier, shift, 2^(shift-1)
    int m1, s1, h1;    // the residual tensor
};
template <bool RELU, bool S32>      // S32: every lane's shift is exactly 32, the high word is the requantised value
__device__ __forceinline__ int4 epilogue16_res1(const uint32_t (&r)[16], const ChannelRq& rq, const int4& res,
                                                const ResidualOne& t) {
    const int sh = rq.s - 32;
    const uint32_t words[4] = {(uint32_t)res.x, (uint32_t)res.y, (uint32_t)res.z, (uint32_t)res.w};
    int q[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int hi = ptx::mad_hi64((int)r[i], rq.m, rq.c64);
        const int a = clamp_i8(S32 ? hi : hi >> sh);
        const uint32_t w = words[i >> 2];
        const int rb = (i & 3) == 0 ? ptx::sext_byte<0>(w) : (i & 3) == 1 ? ptx::sext_byte<1>(w) : (i & 3) == 2 ? ptx::sext_byte<2>(w) : ptx::sext_byte<3>(w);
        q[i] = ((a * t.m0 + t.h0) >> t.s0) + ((rb * t.m1 + t.h1) >> t.s1);
    }
    uint4 o;
    o.x = ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
    o.y = ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
    o.z = ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
    o.w = ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
    if (RELU) {       // on the packed bytes: max(sat8(v), 0) = sat8(max(v, 0))
        o.x = ptx::relu4_s8(o.x); o.y = ptx::relu4_s8(o.y);
        o.z = ptx::relu4_s8(o.z); o.w = ptx::relu4_s8(o.w);
    }
    return make_int4((int)o.x, (int)o.y, (int)o.z, (int)o.w);
}

// Everything an epilogue thread needs to turn 16 accumulator columns into 16 output bytes.
struct EpiThread {
    ChannelRq rq;
    int bias;
    bool all_fast;
    bool valid_o;
    size_t row;        // element offset of (b, o, 0) in the output / residual tensors
};

template <class Params>
__device__ __forceinline__ int4 epilogue16(const Params& p, const EpiThread& e, const uint32_t (&r)[16],
                                           int t, bool in_range) {
    int q[16];
    if (e.all_fast) {
        const int sh = e.rq.s - 32;
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = requant_fast((int)r[i], e.rq.m, e.rq.c64, sh);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = requant_slow((int)r[i], e.rq);
    }
    if (p.terms.n > 0) {
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = clamp_i8(q[i]);
        const size_t idx = e.row + t;
        if (p.terms_fast) {
            int v[16];
            const int m0 = p.terms.mult[0], s0 = p.terms.shift[0];
            const int h0 = 1 << (s0 - 1);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = (q[i] * m0 + h0) >> s0;
            for (int j = 1; j < p.terms.n; ++j) {
                int4 rv = make_int4(0, 0, 0, 0);
                if (in_range) rv = __ldg(reinterpret_cast<const int4*>(p.terms.ptr[j] + idx));
                const int words[4] = {rv.x, rv.y, rv.z, rv.w};
                const int mj = p.terms.mult[j], sj = p.terms.shift[j];
                const int hj = 1 << (sj - 1);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int qv = (int)(int8_t)(words[i >> 2] >> ((i & 3) * 8));
                    v[i] += (qv * mj + hj) >> sj;
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) q[i] = v[i];
            uint4 o;
            o.x = ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
            o.y = ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
            o.z = ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
            o.w = ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
            if (p.relu) {       // on the packed bytes: max(sat8(v), 0) = sat8(max(v, 0))
                o.x = ptx::relu4_s8(o.x); o.y = ptx::relu4_s8(o.y);
                o.z = ptx::relu4_s8(o.z); o.w = ptx::relu4_s8(o.w);
            }
            return make_int4((int)o.x, (int)o.y, (int)o.z, (int)o.w);
        } else {
            long long v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = rescale_term(q[i], p.terms.mult[0], p.terms.shift[0]);
            for (int j = 1; j < p.terms.n; ++j) {
                int4 rv = make_int4(0, 0, 0, 0);
                if (in_range) rv = __ldg(reinterpret_cast<const int4*>(p.terms.ptr[j] + idx));
                const int words[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int qv = (int)(int8_t)(words[i >> 2] >> ((i & 3) * 8));
                    v[i] += rescale_term(qv, p.terms.mult[j], p.terms.shift[j]);
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                long long w = v[i];
                if (p.relu && w < 0) w = 0;
                q[i] = (int)clamp_i8_ll(w);
            }
        }
    } else if (p.relu) {
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = max(q[i], 0);
    }
    int4 out;
    out.x = (int)ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
    out.y = (int)ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
    out.z = (int)ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
    out.w = (int)ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
    return out;
}

}  // namespace tc
}  // namespace qasr
