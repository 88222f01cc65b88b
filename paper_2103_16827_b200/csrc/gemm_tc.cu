// Pointwise (1x1) convolution as an int8 tensor-core GEMM with the fused epilogue.
//
//   acc[o, t] = sum_i W[o, i] * X[b, i, t]          tcgen05.mma kind::i8, accumulator in TMEM
//   y = epilogue(acc + bias)                         requant, residual terms, ReLU, clamp, int8 store
//
// Operands.  A = W tile [128 output channels][64 input channels], K-major, 64-byte swizzle, streamed
// through a ring of TMA stages.  B = X tile [64 input channels][up to 256 frames], MN-major (frames
// are contiguous in the [B][C][T] tensors), 128-byte swizzle.  The whole [C_in][BN] activation tile
// of a work item stays resident in shared memory and is reused by every 128-channel output tile, so
// activations cross L2->SM once per item and only the weights are re-streamed.
//
// Work item = (utterance b, frame tile, group of output-channel tiles); a persistent CTA per SM walks
// the items.  Every CTA visits the output-channel tiles and the K blocks in its own rotated order (the
// integer sum does not care), so that the CTAs do not all pull the same weight block from L2 at once.  Warp roles: warp 0 issues TMA loads, warp 1 owns TMEM and issues the MMAs, warps 2..17
// run the epilogue on a double-buffered accumulator (2 x 256 TMEM columns), so the epilogue of one
// output tile overlaps the MMAs of the next.  Every epilogue warp stages its own [32 channels] x
// [its share of the tile's frames] block in shared memory and writes it with its own TMA store, which
// also clips the ragged edges (frames >= T, channels >= C_out); the epilogue warps never wait for
// one another.
#include <cstdio>
#include <cstring>

#include "qasr_device.cuh"
#include "qasr_host.h"
#include "sm100_ptx.cuh"
#include "tc_epilogue.cuh"

namespace qasr {
namespace tc {

constexpr int BM = 128;            // output channels per MMA tile (TMEM lanes)
// BK = input channels per pipeline block: 128 when C_in allows it (16 KiB per TMA box, 128-byte swizzle
// for the weights), else 64 (8 KiB boxes, 64-byte swizzle). A template parameter of the kernel.
constexpr int MAX_W_STAGES = 8;    // weight ring: as many stages as shared memory leaves room for
constexpr int MAX_KB = 16;         // C_in <= 1024
static_assert(MAX_KB + MAX_W_STAGES + 2 <= 31, "the barriers are initialised by one warp, one lane each");
// Sixteen epilogue warps. As one group, four per 32-channel quarter split a tile's frames; as two groups of eight
// (template parameter GROUPS = 2), group g takes the output tiles of accumulator buffer g and two warps per
// quarter split the frames, so that the fixed part of one tile's epilogue (constants, waits, store issue)
// overlaps the arithmetic of the other tile's.
constexpr int EPI_WARPS = 16;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int ACC_STRIDE = 256;    // TMEM columns between the two accumulator buffers
constexpr int TMEM_COLS = 512;

struct GemmParams {
    int B, C_in, C_out, T;         // T = frames per utterance (input == output length)
    int BN, NC;                    // frames per tile (multiple of 16) and 128-frame chunks per tile
    int tiles_t;                   // frame tiles per utterance
    int m_tiles, m_groups;         // 128-channel output tiles and groups they are split into
    int n_items;
    int w_stages;                  // depth of the weight ring (<= MAX_W_STAGES)
    int w_pair;                    // a weight stage holds two K blocks: every output tile of an item but the first
                                   // (whose blocks are wanted one by one, as the activation blocks arrive) takes one
                                   // barrier round trip and one commit per two K blocks
    int out_bytes;                 // bytes of the output staging area (one block per epilogue warp)
    int stage_w;                   // bytes per staged row of the wider warps (16 * ceil(chunks / warps per quarter))
    const int32_t* bias;
    const int32_t* mult;
    const uint8_t* shift;
    int8_t* y;
    int32_t* y32;
    int relu;
    int terms_fast;                // the residual stage fits 32-bit arithmetic bit for bit (qasr_terms_fit_int32)
    QasrTerms terms;
    unsigned* status;
    QasrPrefetch next;             // constants of the kernel that follows
};

struct SharedTail {
    uint64_t xfull[MAX_KB], xempty[MAX_KB];
    uint64_t wfull[MAX_W_STAGES], wempty[MAX_W_STAGES];
    uint64_t accfull[2], accempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ void item_coords(const GemmParams& p, int item, int& b, int& t0, int& m_lo, int& m_hi) {
    const int mg = item % p.m_groups;
    const int nt = item / p.m_groups;
    b = nt / p.tiles_t;
    t0 = (nt % p.tiles_t) * p.BN;
    const int per = (p.m_tiles + p.m_groups - 1) / p.m_groups;
    m_lo = mg * per;
    m_hi = min(p.m_tiles, m_lo + per);
}

template <int BK, int GROUPS, bool RES1>
__global__ void __launch_bounds__(THREADS, 1)
gemm_i8_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                  const __grid_constant__ CUtensorMap tmXl,
                  const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmYw,
                  const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int W_BLOCK_BYTES = BM * BK;
    constexpr int X_BLOCK_BYTES = BK * 128;     // one (BK channels x 128 frames) swizzled block
    const int W_STAGES = p.w_stages;
    const int W_STAGE_BYTES = p.w_pair ? 2 * W_BLOCK_BYTES : W_BLOCK_BYTES;
    const int KB = p.C_in / BK;
    uint8_t* Xs = smem;                                         // KB * NC blocks of 8 KiB
    uint8_t* Ws = Xs + (size_t)KB * p.NC * X_BLOCK_BYTES;       // W_STAGES stages of 8 KiB
    uint8_t* Os = Ws + W_STAGES * W_STAGE_BYTES;                // [128 channels][BN frames] output staging
    SharedTail* sh = (SharedTail*)(Os + p.out_bytes);

    constexpr int EPI_PARTS = EPI_WARPS / (4 * GROUPS);     // warps per quarter that share one tile
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // one barrier (pair) per thread of warp 2, so that the set-up is not one thread's serial chain
    if (warp == 2) {
        if (lane < MAX_KB) {
            ptx::mbar_init(ptx::smem_u32(&sh->xfull[lane]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->xempty[lane]), 1);
        } else if (lane < MAX_KB + MAX_W_STAGES) {
            ptx::mbar_init(ptx::smem_u32(&sh->wfull[lane - MAX_KB]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->wempty[lane - MAX_KB]), 1);
        } else if (lane < MAX_KB + MAX_W_STAGES + 2) {
            ptx::mbar_init(ptx::smem_u32(&sh->accfull[lane - MAX_KB - MAX_W_STAGES]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->accempty[lane - MAX_KB - MAX_W_STAGES]), EPI_WARPS / GROUPS);
        }
        if (lane == 31) sh->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), TMEM_COLS);
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
        ptx::tma_prefetch_desc(&tmXl);
        ptx::tma_prefetch_desc(&tmY);
        ptx::tma_prefetch_desc(&tmYw);
    }
    if (warp == 2) prefetch_ranges_l2(p.next, lane);
    // everything above touched only this CTA's own state; from here on the previous kernel's output is read
    ptx::grid_dep_launch();
    // griddepcontrol.wait follows inside each role, after the set-up that needs nothing from the previous kernel

    // The producer and the MMA issuer are single threads: one pipeline step costs the latency of their
    // own instruction chains, so both loops carry stage indices, phase bits, barrier addresses and
    // descriptors as running values (no division, no descriptor rebuild per step).
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int NC = p.NC;
            const uint32_t last_w = (uint32_t)(p.BN - 128 * (p.NC - 1));   // frames of the tile's last chunk
            const uint32_t xs_base = ptx::smem_u32(Xs), ws_base = ptx::smem_u32(Ws);
            const uint32_t xfull0 = ptx::smem_u32(&sh->xfull[0]), xempty0 = ptx::smem_u32(&sh->xempty[0]);
            const uint32_t wfull0 = ptx::smem_u32(&sh->wfull[0]), wempty0 = ptx::smem_u32(&sh->wempty[0]);
            int ws = 0;
            uint32_t wph = 1, iph = 1;      // parities to wait for on the "empty" barriers (first pass: free)
            bool ok = true;
            auto issue_w = [&](int m, int kb) {
                ok = ptx::mbar_try(wempty0 + ws * 8, wph) || ptx::mbar_wait(wempty0 + ws * 8, wph, abort_flag, p.status);
                if (!ok) return;
                const uint32_t bar = wfull0 + ws * 8;
                ptx::mbar_expect_tx(bar, W_BLOCK_BYTES);
                ptx::tma_load_2d(ws_base + ws * W_STAGE_BYTES, &tmW, kb * BK, m * BM, bar);
                if (++ws == W_STAGES) { ws = 0; wph ^= 1u; }
            };
            auto issue_w2 = [&](int m, int kb, int kb1) {       // two K blocks into one stage
                ok = ptx::mbar_try(wempty0 + ws * 8, wph) || ptx::mbar_wait(wempty0 + ws * 8, wph, abort_flag, p.status);
                if (!ok) return;
                const uint32_t bar = wfull0 + ws * 8;
                ptx::mbar_expect_tx(bar, 2 * W_BLOCK_BYTES);
                ptx::tma_load_2d(ws_base + ws * W_STAGE_BYTES, &tmW, kb * BK, m * BM, bar);
                ptx::tma_load_2d(ws_base + ws * W_STAGE_BYTES + W_BLOCK_BYTES, &tmW, kb1 * BK, m * BM, bar);
                if (++ws == W_STAGES) { ws = 0; wph ^= 1u; }
            };
            // coordinates of an item; those of the first one are ready before the dependency wait returns
            struct ItemAt { int b, t0, m_lo, mc, rot_m, rot_k; };
            auto locate = [&](int item) {
                ItemAt it;
                int m_hi;
                item_coords(p, item, it.b, it.t0, it.m_lo, m_hi);
                it.mc = m_hi - it.m_lo;
                it.rot_m = it.mc > 0 ? (int)(blockIdx.x % it.mc) : 0;
                it.rot_k = it.mc > 0 ? (int)((blockIdx.x / it.mc) % KB) : 0;
                return it;
            };
            ItemAt at = locate(blockIdx.x < (unsigned)p.n_items ? (int)blockIdx.x : 0);
            ptx::grid_dep_wait();
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, at = locate(item < p.n_items ? item : 0)) {
                const int b = at.b, t0 = at.t0, m_lo = at.m_lo, mc = at.mc, rot_m = at.rot_m, rot_k = at.rot_k;
                if (mc <= 0) continue;
                int kb = rot_k;
                for (int ki = 0; ki < KB && ok; ++ki) {
                    ok = ptx::mbar_try(xempty0 + kb * 8, iph) || ptx::mbar_wait(xempty0 + kb * 8, iph, abort_flag, p.status);
                    if (!ok) break;
                    const uint32_t bar = xfull0 + kb * 8;
                    // the last 128-frame chunk of the tile is loaded only as wide as the tile needs it (a narrower
                    // box keeps the 128-byte row pitch and the swizzle; the bytes behind it are never read)
                    ptx::mbar_expect_tx(bar, (NC - 1) * X_BLOCK_BYTES + BK * last_w);
                    for (int nc = 0; nc < NC - 1; ++nc)
                        ptx::tma_load_3d(xs_base + (uint32_t)(kb * NC + nc) * X_BLOCK_BYTES, &tmX, t0 + nc * 128, kb * BK, b, bar);
                    ptx::tma_load_3d(xs_base + (uint32_t)(kb * NC + NC - 1) * X_BLOCK_BYTES, &tmXl, t0 + (NC - 1) * 128, kb * BK, b, bar);
                    issue_w(m_lo + rot_m, kb);
                    if (++kb == KB) kb = 0;
                }
                int mr = rot_m;
                for (int mi = 1; mi < mc && ok; ++mi) {
                    if (++mr == mc) mr = 0;
                    kb = rot_k;
                    if (p.w_pair) {
                        for (int ki = 0; ki < KB && ok; ki += 2) {
                            const int kb1 = kb + 1 == KB ? 0 : kb + 1;
                            issue_w2(m_lo + mr, kb, kb1);
                            kb = kb1 + 1 == KB ? 0 : kb1 + 1;
                        }
                    } else {
                        for (int ki = 0; ki < KB && ok; ++ki) {
                            issue_w(m_lo + mr, kb);
                            if (++kb == KB) kb = 0;
                        }
                    }
                }
                iph ^= 1u;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // the whole warp walks the loop (all lanes poll the barriers); one elected lane issues
        {
            const uint32_t idesc = ptx::idesc_i8(BM, p.BN, 0, 1);
            // A: K-major rows of BK bytes (swizzle span = BK), 8-row groups 8*BK bytes apart; K advances
            // 32 bytes inside the row. B: MN-major, 128 frames contiguous, 8-channel groups 1024 bytes
            // apart, next 128-frame chunk one block further; K advances 32 channels (4 KiB). Only the
            // start-address field (bits 0..13, 16-byte units) of a descriptor changes from step to step.
            const uint64_t a_desc0 = ptx::smem_desc(0, 16, 8 * BK, BK == 128 ? ptx::SWIZZLE_128B : ptx::SWIZZLE_64B) + (ptx::smem_u32(Ws) >> 4);
            const uint64_t b_desc0 = ptx::smem_desc(0, X_BLOCK_BYTES, 1024, ptx::SWIZZLE_128B) + (ptx::smem_u32(Xs) >> 4);
            const uint32_t x_kb16 = (uint32_t)(p.NC * X_BLOCK_BYTES) >> 4;
            const uint32_t xfull0 = ptx::smem_u32(&sh->xfull[0]), xempty0 = ptx::smem_u32(&sh->xempty[0]);
            const uint32_t wfull0 = ptx::smem_u32(&sh->wfull[0]), wempty0 = ptx::smem_u32(&sh->wempty[0]);
            int ws = 0;
            uint32_t wph = 0, iph = 0, acount = 0;
            bool ok = true;
            ptx::grid_dep_wait();
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                int b, t0, m_lo, m_hi;
                item_coords(p, item, b, t0, m_lo, m_hi);
                if (m_lo >= m_hi) continue;
                const int mc = m_hi - m_lo;
                const int rot_k = (blockIdx.x / mc) % KB;
                for (int mi = 0; mi < mc && ok; ++mi, ++acount) {
                    const int a = acount & 1u;
                    ok = ptx::mbar_wait(ptx::smem_u32(&sh->accempty[a]), ((acount >> 1) & 1u) ^ 1u, abort_flag, p.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + a * ACC_STRIDE;
                    const bool first = mi == 0, last = mi == mc - 1;
                    uint32_t accumulate = 0;
                    int kb = rot_k;
                    if (p.w_pair && !first) {
                        // the activation tile is resident: two K blocks per weight stage
                        for (int ki = 0; ki < KB; ki += 2) {
                            ok = ptx::mbar_try(wfull0 + ws * 8, wph) || ptx::mbar_wait(wfull0 + ws * 8, wph, abort_flag, p.status);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            ptx::tc_fence_after();
                            const int kb1 = kb + 1 == KB ? 0 : kb + 1;
                            const uint64_t ad = a_desc0 + (uint32_t)ws * ((uint32_t)W_STAGE_BYTES >> 4);
                            const uint64_t bd = b_desc0 + (uint32_t)kb * x_kb16;
                            const uint64_t bd1 = b_desc0 + (uint32_t)kb1 * x_kb16;
                            __syncwarp();
                            if (ptx::elect_one()) {
#pragma unroll
                                for (int j = 0; j < BK / 32; ++j)
                                    ptx::mma_i8(d_tmem, ad + 2 * j, bd + 256 * j, idesc, j == 0 ? accumulate : 1u);
#pragma unroll
                                for (int j = 0; j < BK / 32; ++j)
                                    ptx::mma_i8(d_tmem, ad + (W_BLOCK_BYTES >> 4) + 2 * j, bd1 + 256 * j, idesc, 1u);
                                ptx::tc_commit(wempty0 + ws * 8);
                                if (last) { ptx::tc_commit(xempty0 + kb * 8); ptx::tc_commit(xempty0 + kb1 * 8); }
                            }
                            accumulate = 1;
                            if (++ws == W_STAGES) { ws = 0; wph ^= 1u; }
                            kb = kb1 + 1 == KB ? 0 : kb1 + 1;
                        }
                    } else
                    for (int ki = 0; ki < KB; ++ki) {
                        if (first) ok = ptx::mbar_try(xfull0 + kb * 8, iph) || ptx::mbar_wait(xfull0 + kb * 8, iph, abort_flag, p.status);
                        if (ok) ok = ptx::mbar_try(wfull0 + ws * 8, wph) || ptx::mbar_wait(wfull0 + ws * 8, wph, abort_flag, p.status);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint64_t ad = a_desc0 + (uint32_t)ws * ((uint32_t)W_STAGE_BYTES >> 4);
                        const uint64_t bd = b_desc0 + (uint32_t)kb * x_kb16;
                        __syncwarp();
                        if (ptx::elect_one()) {
#pragma unroll
                            for (int j = 0; j < BK / 32; ++j)
                                ptx::mma_i8(d_tmem, ad + 2 * j, bd + 256 * j, idesc, j == 0 ? accumulate : 1u);
                            ptx::tc_commit(wempty0 + ws * 8);
                            if (last) ptx::tc_commit(xempty0 + kb * 8);
                        }
                        accumulate = 1;
                        if (++ws == W_STAGES) { ws = 0; wph ^= 1u; }
                        if (++kb == KB) kb = 0;
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    if (ok && ptx::elect_one()) ptx::tc_commit(ptx::smem_u32(&sh->accfull[a]));
                }
                iph ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 belong to this warp
        const int part = ((warp - 2) >> 2) % EPI_PARTS;   // which share of the tile's 16-frame chunks
        const int egrp = (warp - 2) / (4 * EPI_PARTS);     // which accumulator buffer's tiles (GROUPS == 2)
        const int n_chunks = p.BN >> 4;
        const int c_lo = part * n_chunks / EPI_PARTS;
        const int c_hi = (part + 1) * n_chunks / EPI_PARTS;
        // this warp's staging block: [32 channels][16 * (c_hi - c_lo) frames], dense (the box of its TMA store);
        // tmY's box is 16 * floor(chunks / EPI_PARTS) frames wide, tmYw's one chunk wider
        const int my_w = 16 * (c_hi - c_lo);
        const CUtensorMap* const my_map = my_w == p.stage_w ? &tmYw : &tmY;
        uint8_t* const Ow = Os + (warp - 2) * 32 * p.stage_w;
        uint32_t acount = 0;
        bool ok = true;
        ptx::grid_dep_wait();
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            int b, t0, m_lo, m_hi;
            item_coords(p, item, b, t0, m_lo, m_hi);
            const int mc = m_hi - m_lo;
            for (int mi = 0; mi < mc && ok; ++mi, ++acount) {
                const int m = m_lo + (mi + (int)(blockIdx.x % mc)) % mc;   // the order the producer and MMA warps use
                const int a = acount & 1u;
                if (GROUPS == 2 && a != egrp) continue;         // the other group's tile
                EpiThread e;
                const int o = m * BM + quarter * 32 + lane;
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
                // 0: shift == 32 in every lane, 1: shift >= 32, 2: anything (also residual terms),
                // 3: one residual tensor, 32-bit products, shift >= 32 (its words are fetched a chunk ahead)
                const int mode = RES1 && e.all_fast ? 3
                                 : p.terms.n > 0 ? 2 : (all_s32 ? 0 : (e.all_fast ? 1 : 2));
                ResidualOne ro;
                const int4* res_row = nullptr;      // this thread's residual words for chunk c at res_row[c]
                int4 res_next = make_int4(0, 0, 0, 0);
                if (RES1 && mode == 3) {
                    ro.m0 = p.terms.mult[0]; ro.s0 = p.terms.shift[0]; ro.h0 = 1 << (ro.s0 - 1);
                    ro.m1 = p.terms.mult[1]; ro.s1 = p.terms.shift[1]; ro.h1 = 1 << (ro.s1 - 1);
                    res_row = reinterpret_cast<const int4*>(p.terms.ptr[1] + e.row + t0);
                    if (e.valid_o && c_lo < c_hi && t0 + c_lo * 16 < p.T) res_next = __ldg(res_row + c_lo);
                }
                if (!p.y32) {
                    // this warp's previous TMA store must have finished reading its staging block
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                }
                ok = ptx::mbar_wait(ptx::smem_u32(&sh->accfull[a]), (acount >> 1) & 1u, abort_flag, p.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * ACC_STRIDE;
                uint8_t* orow = Ow + lane * my_w - c_lo * 16;      // chunk c lands at orow + 16 * c

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
                    } else if (RES1 && mode == 3) {
                        const int4 res = res_next;
                        if (e.valid_o && c + 1 < c_hi && t0 + (c + 1) * 16 < p.T) res_next = __ldg(res_row + c + 1);
                        else res_next = make_int4(0, 0, 0, 0);
                        if (all_s32) out = p.relu ? epilogue16_res1<true, true>(r, e.rq, res, ro) : epilogue16_res1<false, true>(r, e.rq, res, ro);
                        else out = p.relu ? epilogue16_res1<true, false>(r, e.rq, res, ro) : epilogue16_res1<false, false>(r, e.rq, res, ro);
                    } else {
                        const int t = t0 + c * 16;
                        out = epilogue16(p, e, r, t, e.valid_o && t < p.T);
                    }
                    *reinterpret_cast<int4*>(orow + c * 16) = out;
                }
                // accumulator drained: hand the TMEM buffer back to the MMA warp
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->accempty[a]));
                if (!p.y32 && my_w > 0) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile(
                            "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                            ::"l"(my_map), "r"(t0 + c_lo * 16), "r"(m * BM + quarter * 32), "r"(b), "r"(ptx::smem_u32(Ow))
                            : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
        }
        // the staging block must outlive the store's read of it; the writes themselves complete with the grid
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
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
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace tc
}  // namespace qasr

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool encode_map(qasr_ctx* ctx, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                       const cuuint64_t* strides_bytes, const cuuint32_t* box, CUtensorMapSwizzle swz) {
    cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    EncodeTiledFn fn = (EncodeTiledFn)ctx->encode_tiled;
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes,
                    box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with code %d", (int)r);
        return false;
    }
    return true;
}

// the same encoder for the other TMA users of the library (uint8 elements)
bool qasr_encode_map_u8(qasr_ctx* ctx, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                        const cuuint64_t* strides_bytes, const cuuint32_t* box, CUtensorMapSwizzle swz) {
    return encode_map(ctx, map, base, rank, dims, strides_bytes, box, swz);
}

static const size_t kSmemLimit = 227 * 1024;

int qasr_gemm_tc_init(qasr_ctx* ctx) {
    cudaError_t e = cudaSuccess;
    auto allow = [&](auto kernel) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
    };
    allow(qasr::tc::gemm_i8_tc_kernel<64, 1, false>); allow(qasr::tc::gemm_i8_tc_kernel<64, 2, false>);
    allow(qasr::tc::gemm_i8_tc_kernel<128, 1, false>); allow(qasr::tc::gemm_i8_tc_kernel<128, 2, false>);
    allow(qasr::tc::gemm_i8_tc_kernel<64, 1, true>); allow(qasr::tc::gemm_i8_tc_kernel<64, 2, true>);
    allow(qasr::tc::gemm_i8_tc_kernel<128, 1, true>); allow(qasr::tc::gemm_i8_tc_kernel<128, 2, true>);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "cudaFuncSetAttribute(gemm_i8_tc_kernel) failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return QASR_OK;
}

// Tile choice: the frame tile BN is an odd multiple of 16 (so the dense [channels][BN] staging tile is
// free of shared-memory bank conflicts for 16-byte row accesses), as wide as the resident activation tile
// allows, and the 128-channel output tiles of one frame tile are split over m_groups CTAs when there
// are fewer frame tiles than SMs. Cost model: rounds of 128-channel tiles per SM x (BN + fixed cost).
static void choose_tiles(int sm_count, int B, int T, int m_tiles, int nc_max, int forced_bn, qasr::tc::GemmParams& p) {
    double best = 1e30;
    // forced_bn: the caller's frame tile (a tuning aid) instead of the search, if the kernel can take it
    const bool forced = forced_bn >= 16 && forced_bn <= 128 * nc_max && forced_bn % 16 == 0;
    for (int bn = forced ? forced_bn : 48; bn <= (forced ? forced_bn : 128 * nc_max); bn += 32) {   // 48, 80, 112, ... : odd multiples of 16
        const int tiles_t = (T + bn - 1) / bn;
        const long long n_tiles = (long long)B * tiles_t;
        for (int g = 1; g <= m_tiles; ++g) {
            const int per = (m_tiles + g - 1) / g;
            if ((m_tiles + per - 1) / per != g) continue;       // would leave an empty group
            const long long rounds = (n_tiles * g + sm_count - 1) / sm_count;
            const double cost = (double)rounds * per * (bn + 40) + (double)rounds * 24 + g;
            if (cost < best) {
                best = cost;
                p.BN = bn; p.tiles_t = tiles_t; p.m_groups = g;
            }
        }
    }
    p.NC = (p.BN + 127) / 128;
}

// Enqueues the pointwise convolution `a` on the tensor cores. The caller has checked that the shape
// qualifies: K == 1, stride == dilation == 1, C_in a multiple of 64 and <= 1024, T a multiple of 16,
// 16-byte aligned tensors.
int qasr_launch_gemm_tc(qasr_ctx* ctx, const QasrConvArgs& a) {
    using namespace qasr::tc;
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.B = a.B; p.C_in = a.C_in; p.C_out = a.C_out; p.T = a.T_out;
    p.m_tiles = (a.C_out + BM - 1) / BM;
    choose_tiles(qasr_grid_slots(ctx), a.B, a.T_out, p.m_tiles, a.C_in <= 512 ? 2 : 1, ctx->force_gemm_bn, p);
    p.n_items = a.B * p.tiles_t * p.m_groups;
    p.bias = a.bias; p.mult = a.mult; p.shift = a.shift; p.y = a.y; p.y32 = a.y_int32; p.relu = a.relu;
    p.terms = a.terms;
    p.terms_fast = qasr_terms_fit_int32(a.terms) ? 1 : 0;
    p.status = ctx->d_status;
    p.next = ctx->prefetch;
    memset(&ctx->prefetch, 0, sizeof(ctx->prefetch));

    // pipeline block, staging tile and weight-ring depth from what shared memory allows
    const int BK = a.C_in % 128 == 0 ? 128 : 64;
    const int n_chunks = p.BN / 16;
    // Two epilogue groups pay where a CTA works through at least two output tiles (of one item or of several) and the
    // wider staging blocks still leave a weight ring of four stages, or where its items have one output tile each, so
    // that every tile waits for a new activation tile and the ring's depth does not matter (measured at B=32:
    // 256->256 7.8 -> 7.5 us, 256->512 11.8 -> 11.1 us, 256->1024 20.2 -> 18.1 us, 512->1024 26.5 -> 24.4 us;
    // 512->512, four tiles per item and a two-stage ring: 13.1 -> 13.3 us, at B=256 75.7 -> 80.8 us, one group kept).
    const int per_item = (p.m_tiles + p.m_groups - 1) / p.m_groups;
    auto layout = [&](int groups, int& stage_w, int& out_bytes, int& w_stages) {
        const int parts = EPI_WARPS / (4 * groups);
        stage_w = 16 * ((n_chunks + parts - 1) / parts);
        out_bytes = a.y ? (EPI_WARPS * 32 * stage_w + 1023) / 1024 * 1024 : 0;
        const size_t fixed_ = 1024 + (size_t)a.C_in * p.NC * 128 + out_bytes + sizeof(SharedTail);
        w_stages = fixed_ >= kSmemLimit ? 0 : (int)((kSmemLimit - fixed_) / (size_t)(BM * BK));
        if (w_stages > MAX_W_STAGES) w_stages = MAX_W_STAGES;
    };
    int GROUPS = 1;
    {
        int sw, ob, ws;
        layout(2, sw, ob, ws);
        const int slots = p.n_items < qasr_grid_slots(ctx) ? p.n_items : qasr_grid_slots(ctx);
        const int tiles_per_cta = (p.n_items + slots - 1) / slots * per_item;
        if (a.y && tiles_per_cta >= 2 && ws >= 2 && (ws >= 4 || (per_item == 1 && tiles_per_cta >= 6))) GROUPS = 2;
    }
    const int EPI_PARTS = EPI_WARPS / (4 * GROUPS);
    layout(GROUPS, p.stage_w, p.out_bytes, p.w_stages);
    const size_t fixed = 1024 + (size_t)a.C_in * p.NC * 128 + p.out_bytes + sizeof(SharedTail);
    if (p.w_stages < 2) return QASR_ERR_SHAPE;
    // two K blocks per weight stage where an item has further output tiles after its first and the ring stays two
    // stages deep
    const int KB = a.C_in / BK;
    // (512->512 at B=32 12.1 -> 11.7 us, at B=256 74.3 -> 70.5 us; the benchmark step moves by 0.25 %: its pointwise
    // layers wait for their epilogues as much as for the MMA warp)
    p.w_pair = KB % 2 == 0 && per_item >= 2 && p.w_stages >= 4 ? 1 : 0;
    if (p.w_pair) p.w_stages /= 2;
    CUtensorMap tmW, tmX, tmXl, tmY, tmYw;
    {
        cuuint64_t dims[2] = {(cuuint64_t)a.C_in, (cuuint64_t)a.C_out};
        cuuint64_t strides[1] = {(cuuint64_t)a.C_in};
        cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
        if (!encode_map(ctx, &tmW, a.w, 2, dims, strides, box, BK == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
            return QASR_ERR_CUDA;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.T, (cuuint64_t)a.C_in, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.T, (cuuint64_t)a.T * a.C_in};
        cuuint32_t box[3] = {128u, (cuuint32_t)BK, 1u};
        if (!encode_map(ctx, &tmX, a.x, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
        box[0] = (cuuint32_t)(p.BN - 128 * (p.NC - 1));     // the last chunk of a tile: only the frames the tile covers
        if (!encode_map(ctx, &tmXl, a.x, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
    }
    if (a.y) {
        cuuint64_t dims[3] = {(cuuint64_t)a.T_out, (cuuint64_t)a.C_out, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.T_out, (cuuint64_t)a.T_out * a.C_out};
        // two box widths: the epilogue warps of a quarter split the tile's 16-frame chunks as evenly as they go
        cuuint32_t box[3] = {(cuuint32_t)p.stage_w, 32u, 1u};
        if (!encode_map(ctx, &tmYw, a.y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
        const int narrow = 16 * (n_chunks / EPI_PARTS);
        box[0] = (cuuint32_t)(narrow > 0 ? narrow : p.stage_w);     // no narrow warps with fewer than EPI_PARTS chunks
        if (!encode_map(ctx, &tmY, a.y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
    } else {
        tmY = tmX;   // unused by the int32-output path
        tmYw = tmX;
    }
    const size_t smem = fixed + (size_t)p.w_stages * (p.w_pair ? 2 : 1) * BM * BK;
    const int grid = p.n_items < qasr_grid_slots(ctx) ? p.n_items : qasr_grid_slots(ctx);
    QasrLaunchScope ls(ctx, QASR_K_GEMM_TC, qasr_conv_macs(a), qasr_conv_bytes(a));
    // the residual instantiation: one residual tensor beside the layer's own output, constants that keep every
    // product inside 32 bits (a block's last layer); everything else runs the kernel without that code
    const bool res1 = a.y && a.terms.n == 2 && p.terms_fast;
    auto launch = [&](auto kernel) {
        return qasr_launch_overlapped(ctx, kernel, dim3(grid), dim3(THREADS), smem, tmW, tmX, tmXl, tmY, tmYw, p);
    };
    cudaError_t e;
    if (BK == 128) {
        if (GROUPS == 2) e = res1 ? launch(gemm_i8_tc_kernel<128, 2, true>) : launch(gemm_i8_tc_kernel<128, 2, false>);
        else e = res1 ? launch(gemm_i8_tc_kernel<128, 1, true>) : launch(gemm_i8_tc_kernel<128, 1, false>);
    } else {
        if (GROUPS == 2) e = res1 ? launch(gemm_i8_tc_kernel<64, 2, true>) : launch(gemm_i8_tc_kernel<64, 2, false>);
        else e = res1 ? launch(gemm_i8_tc_kernel<64, 1, true>) : launch(gemm_i8_tc_kernel<64, 1, false>);
    }
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "gemm_i8_tc_kernel launch failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return QASR_OK;
}
