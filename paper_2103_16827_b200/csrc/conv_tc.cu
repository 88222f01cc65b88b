// Dense K-tap convolution as an implicit int8 GEMM on the tensor cores, with the fused epilogue.
//
//   acc[o, t] = sum_k sum_i W[o, i, k] * X[b, i, t*stride + k*dilation - pad]      (zero outside [0, T))
//   y = epilogue(acc + bias)                  requant, residual terms, ReLU, clamp, int8 store
//
// The GEMM-K dimension is (input channel, tap). A tap shifts the activation operand along time,
// and a shared-memory matrix descriptor can only start on a 16-byte boundary, so the shift must not
// run along the contiguous dimension of the operand tile. Two small preparation kernels therefore
// run first, into caller-provided scratch memory:
//   * the activations [B][C_in][T] are transposed to frame-major rows [B][P][T/P][C_in] (P = stride
//     phases: with stride 2 the even and the odd frames form two planes, so that the frames one tap
//     needs for consecutive outputs are consecutive rows of one plane);
//   * the weights [C_out][C_in][K] are regrouped per tap, [K][C_out][C_in].
// In the main kernel B = a [rows][128 channels] activation stage, K-major with 128-byte swizzle;
// tap k of an output tile is the same stage read from row offset k*dilation (whole 128-byte rows:
// the swizzle is a function of the shared-memory address, so any row offset is a valid descriptor
// start). A = one [128 output channels][128 input channels] weight block of one tap. One activation
// stage therefore feeds K weight blocks, padding comes from the zero fill of TMA loads that start
// before row 0 or end after the last row, and no im2col copy exists anywhere.
//
// Work item = (utterance, frame tile, group of 128-channel output tiles); persistent CTAs walk the
// items. Warp 0 issues TMA loads (activation stages and weight blocks in two rings), warp 1 owns
// TMEM and issues the MMAs, warps 2..17 run the epilogue on a double-buffered accumulator, stage
// each 32-channel quarter in shared memory and write it with one TMA store.
#include <cstdio>
#include <cstring>

#include "qasr_device.cuh"
#include "qasr_host.h"
#include "sm100_ptx.cuh"
#include "tc_epilogue.cuh"

namespace qasr {
namespace tc {

constexpr int CV_BM = 128;            // output channels per MMA tile (TMEM lanes)
constexpr int CV_BK = 128;            // input channels per pipeline block
constexpr int CV_MAX_XS = 3;          // activation stages
constexpr int CV_MAX_WS = 8;          // weight stages
constexpr int CV_EPI_PARTS = 4;
constexpr int CV_EPI_WARPS = 4 * CV_EPI_PARTS;
constexpr int CV_THREADS = 64 + 32 * CV_EPI_WARPS;
constexpr int CV_ACC_STRIDE = 256;
constexpr int CV_TMEM_COLS = 512;
constexpr int CV_W_BLOCK_BYTES = CV_BM * CV_BK;          // one tap's [128 x 128] weight block
// A weight stage holds the blocks of several consecutive taps (ConvParams::w_taps; one TMA box, one barrier
// round trip and one commit per 4 * w_taps MMAs): the issuing warp's fixed cost per round is what this kernel's
// rate depends on.
constexpr int CV_MAX_W_TAPS = 4;

struct ConvParams {
    int B, C_in, C_out, T;         // T = output frames per utterance
    int K, dil, P;                 // taps, dilation, planes (= stride)
    int e0;                        // input offset of tap 0 relative to output frame * stride: -pad
    int row_base;                  // plane row held by stage row 0, relative to the tile's first frame
    int R;                         // rows per plane in an activation stage (multiple of 8, <= 256)
    uint16_t tap_row[128];         // stage row at which tap k of the tile's first output frame starts
    int BN, tiles_t, m_tiles, m_groups, n_items, c_chunks;
    int x_stages, w_stages, x_stage_bytes, out_bytes;
    int w_taps;                    // taps per weight stage
    int dual;                      // the output is also written frame-major [B][T][C_out] (tmYt); its staging
                                   // tiles, one [BN frames][32 channels] per quarter, follow the channel-major ones
    const int32_t* bias;
    const int32_t* mult;
    const uint8_t* shift;
    int8_t* y;
    int32_t* y32;
    int relu;
    int terms_fast;
    QasrTerms terms;
    unsigned* status;
};

struct ConvSharedTail {
    uint64_t xfull[CV_MAX_XS], xempty[CV_MAX_XS];
    uint64_t wfull[CV_MAX_WS], wempty[CV_MAX_WS];
    uint64_t accfull[2], accempty[2];
    uint64_t qbar[4];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ void conv_item_coords(const ConvParams& p, int item, int& b, int& t0, int& m_lo, int& m_hi) {
    const int mg = item % p.m_groups;
    const int nt = item / p.m_groups;
    b = nt / p.tiles_t;
    t0 = (nt % p.tiles_t) * p.BN;
    const int per = (p.m_tiles + p.m_groups - 1) / p.m_groups;
    m_lo = mg * per;
    m_hi = min(p.m_tiles, m_lo + per);
}

__global__ void __launch_bounds__(CV_THREADS, 1)
conv_i8_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                  const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmYt,
                  const ConvParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int XS = p.x_stages, WS = p.w_stages;
    uint8_t* Xs = smem;                                          // XS stages of P * R rows of 128 bytes
    uint8_t* Ws = Xs + (size_t)XS * p.x_stage_bytes;             // WS stages of 16 KiB
    const int W_TAPS = p.w_taps;
    const uint32_t W_STAGE_BYTES = (uint32_t)W_TAPS * CV_W_BLOCK_BYTES;
    uint8_t* Os = Ws + (size_t)WS * W_STAGE_BYTES;            // [128 channels][BN frames] output staging
    ConvSharedTail* sh = (ConvSharedTail*)(Os + p.out_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // one barrier (pair) per thread of warp 2, so that the set-up is not one thread's serial chain
    if (warp == 2) {
        if (lane < CV_MAX_XS) {
            ptx::mbar_init(ptx::smem_u32(&sh->xfull[lane]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->xempty[lane]), 1);
        } else if (lane < CV_MAX_XS + CV_MAX_WS) {
            ptx::mbar_init(ptx::smem_u32(&sh->wfull[lane - CV_MAX_XS]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->wempty[lane - CV_MAX_XS]), 1);
        } else if (lane < CV_MAX_XS + CV_MAX_WS + 2) {
            ptx::mbar_init(ptx::smem_u32(&sh->accfull[lane - CV_MAX_XS - CV_MAX_WS]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->accempty[lane - CV_MAX_XS - CV_MAX_WS]), CV_EPI_WARPS);
        } else if (lane < CV_MAX_XS + CV_MAX_WS + 6) {
            ptx::mbar_init(ptx::smem_u32(&sh->qbar[lane - CV_MAX_XS - CV_MAX_WS - 2]), CV_EPI_PARTS);
        }
        if (lane == 31) sh->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), CV_TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;

    if (threadIdx.x == 0) {   // the tensor maps are kernel parameters: fetch them while the previous kernel drains
        ptx::tma_prefetch_desc(&tmW);
        ptx::tma_prefetch_desc(&tmX);
        ptx::tma_prefetch_desc(&tmY);
        if (p.dual) ptx::tma_prefetch_desc(&tmYt);
    }
    // everything above overlaps the tail of the previous kernel; its results are needed from here on
    ptx::grid_dep_launch();
    // griddepcontrol.wait follows inside each role, after the set-up that needs nothing from the previous kernel

    // The producer and the MMA issuer are single threads, so the time of one pipeline step is the
    // latency of their own instruction chains: the loops below carry stage indices, phase bits,
    // barrier addresses and descriptors as running values (no division, no address rebuild per step).
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int K = p.K, P = p.P, c_chunks = p.c_chunks, row_base = p.row_base;
            const uint32_t x_stage_bytes = (uint32_t)p.x_stage_bytes, plane_bytes = (uint32_t)p.R * 128u;
            const uint32_t xs_base = ptx::smem_u32(Xs), ws_base = ptx::smem_u32(Ws);
            const uint32_t xfull0 = ptx::smem_u32(&sh->xfull[0]), xempty0 = ptx::smem_u32(&sh->xempty[0]);
            const uint32_t wfull0 = ptx::smem_u32(&sh->wfull[0]), wempty0 = ptx::smem_u32(&sh->wempty[0]);
            int ws = 0, xs = 0;
            uint32_t wph = 1, xph = 1;      // parity to wait for on the "empty" barriers (first pass: free)
            bool ok = true;
            int b, t0, m_lo, m_hi;      // the first item's coordinates are ready before the dependency wait returns
            conv_item_coords(p, blockIdx.x < (unsigned)p.n_items ? (int)blockIdx.x : 0, b, t0, m_lo, m_hi);
            ptx::grid_dep_wait();
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                if (item != (int)blockIdx.x) conv_item_coords(p, item, b, t0, m_lo, m_hi);
                for (int m = m_lo; m < m_hi && ok; ++m) {
                    for (int cc = 0; cc < c_chunks && ok; ++cc) {
                        ok = ptx::mbar_try(xempty0 + xs * 8, xph) || ptx::mbar_wait(xempty0 + xs * 8, xph, abort_flag, p.status);
                        if (!ok) break;
                        const uint32_t xbar = xfull0 + xs * 8;
                        ptx::mbar_expect_tx(xbar, x_stage_bytes);
                        for (int pl = 0; pl < P; ++pl)
                            ptx::tma_load_3d(xs_base + xs * x_stage_bytes + pl * plane_bytes, &tmX,
                                             cc * CV_BK, t0 + row_base, b * P + pl, xbar);
                        if (++xs == XS) { xs = 0; xph ^= 1u; }
                        for (int k = 0; k < K; k += W_TAPS) {     // taps >= K of the last box arrive as zeros, never used
                            ok = ptx::mbar_try(wempty0 + ws * 8, wph) || ptx::mbar_wait(wempty0 + ws * 8, wph, abort_flag, p.status);
                            if (!ok) break;
                            const uint32_t wbar = wfull0 + ws * 8;
                            ptx::mbar_expect_tx(wbar, W_STAGE_BYTES);
                            ptx::tma_load_3d(ws_base + ws * W_STAGE_BYTES, &tmW, cc * CV_BK, m * CV_BM, k, wbar);
                            if (++ws == WS) { ws = 0; wph ^= 1u; }
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // the whole warp walks the loop (all lanes poll the barriers); one elected lane issues
        {
            const uint32_t idesc = ptx::idesc_i8(CV_BM, p.BN, 0, 0);
            const int K = p.K, c_chunks = p.c_chunks;
            const int ksteps_last = min(CV_BK / 32, (p.C_in - (c_chunks - 1) * CV_BK + 31) / 32);
            const uint32_t x_stage16 = (uint32_t)p.x_stage_bytes >> 4;
            // both operands K-major: rows of 128 bytes, 8-row groups 1024 bytes apart; the start address
            // field (bits 0..13, in 16-byte units) is the only part of a descriptor that changes
            const uint64_t desc0 = ptx::smem_desc(0, 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t a_desc0 = desc0 + (ptx::smem_u32(Ws) >> 4);
            const uint64_t b_desc0 = desc0 + (ptx::smem_u32(Xs) >> 4);
            const uint32_t xfull0 = ptx::smem_u32(&sh->xfull[0]), xempty0 = ptx::smem_u32(&sh->xempty[0]);
            const uint32_t wfull0 = ptx::smem_u32(&sh->wfull[0]), wempty0 = ptx::smem_u32(&sh->wempty[0]);
            int ws = 0, xs = 0;
            uint32_t wph = 0, xph = 0, acount = 0;
            bool ok = true;
            ptx::grid_dep_wait();
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                int b, t0, m_lo, m_hi;
                conv_item_coords(p, item, b, t0, m_lo, m_hi);
                for (int m = m_lo; m < m_hi && ok; ++m, ++acount) {
                    const int a = acount & 1u;
                    ok = ptx::mbar_wait(ptx::smem_u32(&sh->accempty[a]), ((acount >> 1) & 1u) ^ 1u, abort_flag, p.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + a * CV_ACC_STRIDE;
                    uint32_t accumulate = 0;
                    for (int cc = 0; cc < c_chunks && ok; ++cc) {
                        ok = ptx::mbar_try(xfull0 + xs * 8, xph) || ptx::mbar_wait(xfull0 + xs * 8, xph, abort_flag, p.status);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        const uint64_t b_stage = b_desc0 + (uint32_t)xs * x_stage16;
                        const int ksteps = cc == c_chunks - 1 ? ksteps_last : CV_BK / 32;
                        for (int k = 0; k < K; k += W_TAPS) {
                            ok = ptx::mbar_try(wfull0 + ws * 8, wph) || ptx::mbar_wait(wfull0 + ws * 8, wph, abort_flag, p.status);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            ptx::tc_fence_after();
                            uint64_t ad = a_desc0 + (uint32_t)ws * (W_STAGE_BYTES >> 4);
                            const int taps_here = min(W_TAPS, K - k);
                            if (ptx::elect_one()) {
                                for (int u = 0; u < taps_here; ++u, ad += CV_W_BLOCK_BYTES >> 4) {
                                    const uint64_t bd = b_stage + (uint32_t)p.tap_row[k + u] * 8u;      // whole 128-byte rows
#pragma unroll
                                    for (int j = 0; j < CV_BK / 32; ++j) {
                                        if (j < ksteps)
                                            ptx::mma_i8(d_tmem, ad + 2 * j, bd + 2 * j, idesc, (u | j) == 0 ? accumulate : 1u);   // 32 channels further
                                    }
                                }
                                ptx::tc_commit(wempty0 + ws * 8);
                            }
                            accumulate = 1;
                            if (++ws == WS) { ws = 0; wph ^= 1u; }
                        }
                        if (ok && ptx::elect_one()) ptx::tc_commit(xempty0 + xs * 8);
                        if (++xs == XS) { xs = 0; xph ^= 1u; }
                    }
                    if (ok && ptx::elect_one()) ptx::tc_commit(ptx::smem_u32(&sh->accfull[a]));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 belong to this warp
        const int part = (warp - 2) >> 2;             // which share of the tile's 16-frame chunks
        const int n_chunks = p.BN >> 4;
        const int c_lo = part * n_chunks / CV_EPI_PARTS;
        const int c_hi = (part + 1) * n_chunks / CV_EPI_PARTS;
        const bool issuer = part == 0 && lane == 0;   // issues this quarter's TMA stores
        uint8_t* Oq = Os + quarter * 32 * p.BN;       // [32 channels][BN] dense staging sub-tile
        uint8_t* Otq = Os + (CV_BM + quarter * 32) * p.BN;   // [BN frames][32 channels], the frame-major twin
        uint32_t acount = 0, qcount = 0;
        bool ok = true;
        auto quarter_sync = [&]() -> bool {
            __syncwarp();
            const uint32_t bar = ptx::smem_u32(&sh->qbar[quarter]);
            if (lane == 0) ptx::mbar_arrive(bar);
            const bool r = ptx::mbar_wait(bar, qcount & 1u, abort_flag, p.status);
            ++qcount;
            return __all_sync(0xffffffffu, r);
        };
        ptx::grid_dep_wait();
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            int b, t0, m_lo, m_hi;
            conv_item_coords(p, item, b, t0, m_lo, m_hi);
            for (int m = m_lo; m < m_hi && ok; ++m, ++acount) {
                const int a = acount & 1u;
                EpiThread e;
                const int o = m * CV_BM + quarter * 32 + lane;
                e.valid_o = o < p.C_out;
                e.rq.m = 0; e.rq.s = 32; e.rq.c64 = 0; e.rq.fast = 1;
                e.bias = 0;
                if (e.valid_o) {
                    e.bias = p.bias ? __ldg(p.bias + o) : 0;
                    if (!p.y32) {
                        int mm, ss;
                        load_rq(p.mult, p.shift, o, mm, ss, p.status);
                        e.rq = make_rq(e.bias, mm, ss);
                    }
                }
                e.all_fast = __all_sync(0xffffffffu, e.rq.fast != 0);
                const bool all_s32 = __all_sync(0xffffffffu, e.rq.s == 32);
                e.row = ((size_t)b * p.C_out + (e.valid_o ? o : 0)) * p.T;
                const int mode = p.terms.n > 0 ? 2 : (all_s32 ? 0 : (e.all_fast ? 1 : 2));
                if (!p.y32) {
                    // the previous TMA store of this quarter must have finished reading the staging tile
                    if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    ok = quarter_sync();
                    if (!ok) break;
                }
                ok = ptx::mbar_wait(ptx::smem_u32(&sh->accfull[a]), (acount >> 1) & 1u, abort_flag, p.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * CV_ACC_STRIDE;
                uint8_t* orow = Oq + lane * p.BN;

                for (int c = c_lo; c < c_hi; ++c) {
                    uint32_t r[16];
                    __syncwarp();
                    ptx::tmem_ld16(taddr + c * 16, r);
                    ptx::tmem_ld_wait(r);
                    if (p.y32) {
                        const int t = t0 + c * 16;
                        if (e.valid_o && t < p.T) {     // T is a multiple of 16: all-or-nothing
                            int4* dst = reinterpret_cast<int4*>(p.y32 + e.row + t);
#pragma unroll
                            for (int v = 0; v < 4; ++v)
                                dst[v] = make_int4((int)r[4 * v] + e.bias, (int)r[4 * v + 1] + e.bias,
                                                   (int)r[4 * v + 2] + e.bias, (int)r[4 * v + 3] + e.bias);
                        }
                        continue;
                    }
                    int4 out;
                    if (mode == 0) {
                        out = p.relu ? requant16<0, true>(r, e.rq) : requant16<0, false>(r, e.rq);
                    } else if (mode == 1) {
                        out = p.relu ? requant16<1, true>(r, e.rq) : requant16<1, false>(r, e.rq);
                    } else {
                        const int t = t0 + c * 16;
                        out = epilogue16(p, e, r, t, e.valid_o && t < p.T);
                    }
                    *reinterpret_cast<int4*>(orow + c * 16) = out;
                    if (p.dual) {
                        // the same 16 frames of this lane's channel, one byte per frame row: the 32 lanes of a
                        // warp fill 32 consecutive bytes of a row per store (one wavefront)
                        uint8_t* const ot = Otq + c * 16 * 32 + lane;
                        const uint32_t wd[4] = {(uint32_t)out.x, (uint32_t)out.y, (uint32_t)out.z, (uint32_t)out.w};
#pragma unroll
                        for (int i = 0; i < 16; ++i) ot[i * 32] = (uint8_t)(wd[i >> 2] >> (8 * (i & 3)));
                    }
                }
                // accumulator drained: hand the TMEM buffer back to the MMA warp
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->accempty[a]));
                if (!p.y32) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    ok = quarter_sync();
                    if (!ok) break;
                    if (issuer) {
                        asm volatile(
                            "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                            ::"l"(&tmY), "r"(t0), "r"(m * CV_BM + quarter * 32), "r"(b), "r"(ptx::smem_u32(Oq))
                            : "memory");
                        if (p.dual)     // box: 32 channels x BN frames; frames >= T and channels >= C_out are clipped
                            asm volatile(
                                "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                                ::"l"(&tmYt), "r"(m * CV_BM + quarter * 32), "r"(t0), "r"(b), "r"(ptx::smem_u32(Otq))
                                : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
        }
        // the staging tile must outlive the store's read of it; the writes themselves complete with the grid
        if (issuer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }

    // ---------------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (*abort_flag) {          // uniform after the barrier
        // a wait gave up: give copies that may still be in flight a bounded time to land
        if (threadIdx.x == 0)
            for (int i = 0; i < 64; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, CV_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------
// preparation kernels
// ------------------------------------------------------------------------------------------

// x [B][C][T] (frames contiguous) -> xt [B][P][T/P][C] (channels contiguous); frame f goes to plane
// f % P, row f / P. A block moves 64 channels x 128 frames: coalesced 128-byte row reads, 4x4 byte
// transposes in registers, a shared-memory tile, coalesced 64-byte row writes.
constexpr int TR_C = 64, TR_F = 128;
__global__ void __launch_bounds__(256)
transpose_frames_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ xt, int C, int T, int P, int Tp) {
    __shared__ uint32_t tile[TR_F][TR_C / 4 + 1];
    const int b = blockIdx.z;
    const int c0 = blockIdx.y * TR_C, f0 = blockIdx.x * TR_F;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int f = f0 + 4 * lane;
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        const int c = c0 + 8 * warp + 4 * g;
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            w[i] = (c + i < C && f < T) ? __ldg(reinterpret_cast<const uint32_t*>(x + ((size_t)b * C + c + i) * T + f)) : 0u;
        const uint32_t t0 = __byte_perm(w[0], w[1], 0x5140), t1 = __byte_perm(w[2], w[3], 0x5140);
        const uint32_t t2 = __byte_perm(w[0], w[1], 0x7362), t3 = __byte_perm(w[2], w[3], 0x7362);
        tile[4 * lane + 0][2 * warp + g] = __byte_perm(t0, t1, 0x5410);
        tile[4 * lane + 1][2 * warp + g] = __byte_perm(t0, t1, 0x7632);
        tile[4 * lane + 2][2 * warp + g] = __byte_perm(t2, t3, 0x5410);
        tile[4 * lane + 3][2 * warp + g] = __byte_perm(t2, t3, 0x7632);
    }
    __syncthreads();
    const int word = threadIdx.x & 15;
#pragma unroll
    for (int it = 0; it < TR_F / 16; ++it) {
        const int row = (threadIdx.x >> 4) + 16 * it;
        const int fr = f0 + row;
        const int c = c0 + 4 * word;
        if (fr < T && c < C) {
            const int pl = P == 1 ? 0 : (fr & 1), r = P == 1 ? fr : (fr >> 1);
            *reinterpret_cast<uint32_t*>(xt + (((size_t)b * P + pl) * Tp + r) * C + c) = tile[row][word];
        }
    }
}

// w [C_out][C_in][K] -> wt [K][C_out][C_in]; one thread moves 4 input channels of one output channel.
__global__ void __launch_bounds__(256)
regroup_weights_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ wt, int C_out, int C_in, int K) {
    const size_t quad = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // index of (o, c / 4)
    const size_t n_quads = (size_t)C_out * (C_in / 4);
    if (quad >= n_quads) return;
    const int8_t* src = w + quad * 4 * K;
    for (int k = 0; k < K; ++k) {
        const uint32_t v = (uint32_t)(uint8_t)__ldg(src + k) | ((uint32_t)(uint8_t)__ldg(src + K + k) << 8) |
                           ((uint32_t)(uint8_t)__ldg(src + 2 * K + k) << 16) | ((uint32_t)(uint8_t)__ldg(src + 3 * K + k) << 24);
        *reinterpret_cast<uint32_t*>(wt + (size_t)k * C_out * C_in + quad * 4) = v;
    }
}

}  // namespace tc
}  // namespace qasr

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
bool qasr_encode_map_u8(qasr_ctx* ctx, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                        const cuuint64_t* strides_bytes, const cuuint32_t* box, CUtensorMapSwizzle swz);

static const size_t kConvSmemLimit = 227 * 1024;

int qasr_conv_tc_init(qasr_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(qasr::tc::conv_i8_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kConvSmemLimit);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "cudaFuncSetAttribute(conv_i8_tc_kernel) failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return QASR_OK;
}

static inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// Scratch bytes the tensor-core path of a dense convolution needs (transposed input + regrouped weights).
size_t qasr_conv_tc_input_bytes(int B, int C_in, int T, int stride) {
    const int Tp = (T + stride - 1) / stride;
    return up256((size_t)B * stride * Tp * C_in);
}
size_t qasr_conv_tc_weight_bytes(int C_in, int C_out, int K) { return up256((size_t)K * C_out * C_in); }
size_t qasr_conv_tc_scratch_bytes(int B, int C_in, int C_out, int T, int K, int stride) {
    return qasr_conv_tc_input_bytes(B, C_in, T, stride) + qasr_conv_tc_weight_bytes(C_in, C_out, K);
}

// Geometry of the activation stage for a frame tile of BN outputs; false if it does not fit a TMA box.
static bool stage_rows(int K, int stride, int dil, int BN, int& e0, int& row_base, int& R) {
    const int pad = dil * (K - 1) / 2;
    e0 = -pad;
    auto fdiv = [&](int e) { return stride == 1 ? e : (e >> 1); };
    row_base = fdiv(e0);
    const int last = fdiv(e0 + (K - 1) * dil);
    R = BN + (last - row_base);
    R = (R + 7) / 8 * 8;
    return R <= 256;
}

// Enqueues the dense convolution `a` on the tensor cores: returns 1 if it did, 0 if the shape does not
// qualify (the caller then uses the generic kernel), or a negative error code.
int qasr_launch_conv_tc(qasr_ctx* ctx, const QasrConvArgs& a) {
    using namespace qasr::tc;
    if (!a.scratch) return 0;
    if (a.C_in % 16 != 0 || a.T % 16 != 0 || a.T_out % 16 != 0 || a.T_out < 16) return 0;
    if (a.K > 127 || a.C_in > 65535) return 0;
    const int P = a.stride;
    const int Tp = (a.T + P - 1) / P;
    const size_t xt_bytes = up256((size_t)a.B * P * Tp * a.C_in);
    const size_t wt_bytes = up256((size_t)a.K * a.C_out * a.C_in);
    if (a.scratch_bytes < xt_bytes + (a.wt ? 0 : wt_bytes)) return 0;
    // the frame-major second output: int8 results, whole 16-byte rows
    const bool dual = a.yt && a.y && a.C_out % 16 == 0 && ((uintptr_t)a.yt & 15u) == 0;

    ConvParams p;
    memset(&p, 0, sizeof(p));
    p.B = a.B; p.C_in = a.C_in; p.C_out = a.C_out; p.T = a.T_out;
    p.K = a.K; p.dil = a.dilation; p.P = P;
    p.m_tiles = (a.C_out + CV_BM - 1) / CV_BM;
    p.c_chunks = (a.C_in + CV_BK - 1) / CV_BK;

    // Frame tile: an odd multiple of 16 (conflict-free staging rows), as wide as the stage box allows;
    // output-channel tiles are split over m_groups CTAs when there are few frame tiles.
    // Cost: rounds x tiles per group x (weight block time ~ max(BN, 176) + activation share).
    double best = 1e30;
    for (int bn = 48; bn <= 240; bn += 32) {
        int e0, rb, R;
        if (!stage_rows(a.K, a.stride, a.dilation, bn, e0, rb, R)) break;
        const int tiles_t = (a.T_out + bn - 1) / bn;
        const long long n_tiles = (long long)a.B * tiles_t;
        for (int g = 1; g <= p.m_tiles; ++g) {
            const int per = (p.m_tiles + g - 1) / g;
            if ((p.m_tiles + per - 1) / per != g) continue;
            const long long rounds = (n_tiles * g + qasr_grid_slots(ctx) - 1) / qasr_grid_slots(ctx);
            const double blk = (bn > 176 ? bn : 176) + (double)R * P / a.K;
            const double cost = (double)rounds * per * blk + g * 1e-3;
            if (cost < best) {
                best = cost;
                p.BN = bn; p.tiles_t = tiles_t; p.m_groups = g;
                p.e0 = e0; p.row_base = rb; p.R = R;
            }
        }
    }
    if (best >= 1e30) return 0;
    p.n_items = a.B * p.tiles_t * p.m_groups;
    p.bias = a.bias; p.mult = a.mult; p.shift = a.shift; p.y = a.y; p.y32 = a.y_int32; p.relu = a.relu;
    p.terms = a.terms;
    p.terms_fast = qasr_terms_fit_int32(a.terms) ? 1 : 0;
    p.status = ctx->d_status;

    for (int k = 0; k < a.K; ++k) {
        // input offset of tap k; with two planes, frame e lies in plane e mod 2 at row floor(e / 2)
        const int e = p.e0 + k * a.dilation;
        const int plane = P == 1 ? 0 : (e & 1), row = P == 1 ? e : (e >> 1);
        p.tap_row[k] = (uint16_t)(plane * p.R + (row - p.row_base));
    }
    p.x_stage_bytes = P * p.R * 128;
    p.dual = dual ? 1 : 0;
    p.out_bytes = a.y ? ((dual ? 2 : 1) * CV_BM * p.BN + 1023) / 1024 * 1024 : 0;
    const size_t fixed = 1024 + p.out_bytes + sizeof(ConvSharedTail);
    p.x_stages = 3;
    long long room = (long long)kConvSmemLimit - (long long)fixed - (long long)p.x_stages * p.x_stage_bytes;
    if (room < 6LL * CV_W_BLOCK_BYTES) {
        p.x_stages = 2;
        room = (long long)kConvSmemLimit - (long long)fixed - (long long)p.x_stages * p.x_stage_bytes;
    }
    if (room < 3LL * CV_W_BLOCK_BYTES) return 0;
    // taps per weight stage: two where that leaves a ring of at least three stages (measured on 768 -> 768, K = 13,
    // B = 64: 2306 TOP/s with one tap per stage, 2709 with two, 2725 / 2703 with three / four)
    const int blocks = (int)(room / CV_W_BLOCK_BYTES);
    p.w_taps = blocks >= 6 ? 2 : 1;
    if (p.w_taps > a.K) p.w_taps = a.K;
    p.w_stages = blocks / p.w_taps;
    if (p.w_stages > CV_MAX_WS) p.w_stages = CV_MAX_WS;

    int8_t* xt = (int8_t*)a.scratch;
    int8_t* wt = a.wt ? (int8_t*)a.wt : xt + xt_bytes;
    CUtensorMap tmW, tmX, tmY, tmYt;
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.C_in, (cuuint64_t)a.C_out, (cuuint64_t)a.K};
        cuuint64_t strides[2] = {(cuuint64_t)a.C_in, (cuuint64_t)a.C_in * a.C_out};
        cuuint32_t box[3] = {(cuuint32_t)CV_BK, (cuuint32_t)CV_BM, (cuuint32_t)p.w_taps};
        if (!qasr_encode_map_u8(ctx, &tmW, wt, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.C_in, (cuuint64_t)Tp, (cuuint64_t)a.B * P};
        cuuint64_t strides[2] = {(cuuint64_t)a.C_in, (cuuint64_t)a.C_in * Tp};
        cuuint32_t box[3] = {(cuuint32_t)CV_BK, (cuuint32_t)p.R, 1u};
        if (!qasr_encode_map_u8(ctx, &tmX, xt, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
    }
    if (a.y) {
        cuuint64_t dims[3] = {(cuuint64_t)a.T_out, (cuuint64_t)a.C_out, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.T_out, (cuuint64_t)a.T_out * a.C_out};
        cuuint32_t box[3] = {(cuuint32_t)p.BN, 32u, 1u};
        if (!qasr_encode_map_u8(ctx, &tmY, a.y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
    } else {
        tmY = tmX;   // unused by the int32-output path
    }
    tmYt = tmY;      // unused without the second output
    if (dual) {
        cuuint64_t dims[3] = {(cuuint64_t)a.C_out, (cuuint64_t)a.T_out, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.C_out, (cuuint64_t)a.C_out * a.T_out};
        cuuint32_t box[3] = {32u, (cuuint32_t)p.BN, 1u};
        if (!qasr_encode_map_u8(ctx, &tmYt, a.yt, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
    }

    if (!a.xt_ready) {
        QasrLaunchScope ls(ctx, QASR_K_CONV_PREP, 0, 2.0 * a.B * a.C_in * a.T);
        dim3 grid((a.T + TR_F - 1) / TR_F, (a.C_in + TR_C - 1) / TR_C, a.B);
        transpose_frames_kernel<<<grid, 256, 0, ctx->stream>>>(a.x, xt, a.C_in, a.T, P, Tp);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) {
            snprintf(ctx->err, sizeof(ctx->err), "transpose_frames_kernel launch failed: %s", cudaGetErrorString(e));
            return QASR_ERR_CUDA;
        }
    }
    if (!(a.wt && a.wt_ready)) {
        QasrLaunchScope ls(ctx, QASR_K_CONV_PREP, 0, 2.0 * a.K * a.C_out * a.C_in);
        const size_t n_quads = (size_t)a.C_out * (a.C_in / 4);
        regroup_weights_kernel<<<(unsigned)((n_quads + 255) / 256), 256, 0, ctx->stream>>>(a.w, wt, a.C_out, a.C_in, a.K);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) {
            snprintf(ctx->err, sizeof(ctx->err), "regroup_weights_kernel launch failed: %s", cudaGetErrorString(e));
            return QASR_ERR_CUDA;
        }
    }
    const size_t smem = fixed + (size_t)p.x_stages * p.x_stage_bytes + (size_t)p.w_stages * p.w_taps * CV_W_BLOCK_BYTES;
    const int grid = p.n_items < qasr_grid_slots(ctx) ? p.n_items : qasr_grid_slots(ctx);
    QasrLaunchScope ls(ctx, QASR_K_CONV_TC, qasr_conv_macs(a), qasr_conv_bytes(a));
    ctx->hold_early_launch = ctx->grid_cap > 0;      // a side branch shares the GPU
    cudaError_t e = qasr_launch_overlapped(ctx, conv_i8_tc_kernel, dim3(grid), dim3(CV_THREADS), smem, tmW, tmX, tmY, tmYt, p);
    ctx->hold_early_launch = false;
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "conv_i8_tc_kernel launch failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    ctx->yt_written = dual;
    return 1;
}
