// Depthwise K-tap convolution on the tensor cores: one banded (Toeplitz) int8 GEMM per channel.
//
// The dp4a rate of the SM caps a CUDA-core depthwise kernel far below the HBM roofline for K >= 39,
// so the taps are applied by tcgen05.mma instead.  For channel c
//
//     D[r, n] = sum_k A[r, k] * Bt[n, k]
//
//   r  = window (frame tile i, utterance b): 128 windows form the M dimension of one MMA tile,
//   A[r, k]  = x[b, c, i*NT*stride - padL + k]          the window's input bytes (zero outside [0, T)),
//   Bt[n, k] = w[c, (k - n*stride - lead) / dilation]   the taps laid along a band, zero elsewhere,
//   D[r, n]  = accumulator of output frame i*NT + n.
//
// A is K-major with the 128-byte swizzle and comes straight from the activation tensor by TMA: one box
// of [utterances][128 bytes] per frame tile and 128-byte K block, whose out-of-range frames arrive as
// zeros, which is exactly the convolution's padding.  The band makes most of Bt zero, so the NT outputs
// of a tile are produced in sub-blocks of up to 128 columns (64 when shared memory is short): every
// sub-block multiplies the same small band matrix (b_rows x Kspan bytes, K-major, 128-byte swizzle like
// A, written by CUDA-core warps from the channel's taps) with the slice of A that starts at its first
// input byte.  Stride 2 and dilation 2 only move the band.
//
// Warp roles: 2 x 4 builder warps fill the two stages (a few threads issue the TMA loads of A, all build
// Bt) while the MMA warp issues the current stage and 8 epilogue warps requantise the previous
// accumulator (per-channel scalar constants) and store 16 output frames per thread and step.  The taps
// of a group's next item are fetched one item ahead (the first ones before the dependency wait): they
// are constants of the layer whose first touch comes from DRAM.  The first item of each builder group is
// started differently: its band depends on constants only and is built without waiting for the previous
// kernel, and its window loads are issued by the epilogue warps (idle at that point), one box per warp
// side by side, as soon as their dependency wait returns.
#include <cstdio>
#include <cstring>

#include "qasr_device.cuh"
#include "qasr_host.h"
#include "sm100_ptx.cuh"

bool qasr_encode_map_u8(qasr_ctx* ctx, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                        const cuuint64_t* strides_bytes, const cuuint32_t* box, CUtensorMapSwizzle swz);

namespace qasr {
namespace dwtc {

constexpr int BUILD_GROUP_WARPS = 4;
constexpr int BUILD_GROUP_THREADS = 32 * BUILD_GROUP_WARPS;
constexpr int BUILD_WARPS = 2 * BUILD_GROUP_WARPS;   // two groups, one per stage
// Two groups of epilogue warps, one per accumulator buffer: group g requantises every second item. While
// one group sits in the fixed part of an item (constants, barrier waits, store issue) the other one computes.
constexpr int EPI_GROUPS = 2;
constexpr int EPI_GROUP_WARPS = 8;
constexpr int EPI_WARPS = EPI_GROUPS * EPI_GROUP_WARPS;
constexpr int EPI_PARTS = EPI_GROUP_WARPS / 4;   // warps of a group per 32-lane quarter; they split the 16-column chunks
constexpr int MMA_WARP = BUILD_WARPS + EPI_WARPS;
constexpr int THREADS = 32 * (BUILD_WARPS + EPI_WARPS + 1);
constexpr int TMEM_COLS = 512;
constexpr int ACC_STRIDE = 256;
constexpr int A_KBLOCK_BYTES = 128 * 128;    // one 128-byte K block of all 128 windows, swizzled
constexpr int LINE_WORDS = 64;               // tap line: (K-1)*dilation + 1 + 32 bytes <= 240
constexpr int MAX_SB = 4;

struct Params {
    const int8_t* w;
    const int32_t* mult;
    const uint8_t* shift;
    int8_t* y;
    int B, C, T, T_out, K, stride, dil;
    int NT, tiles;
    int rows_b;                      // utterances per box = min(B, 128)
    int tpm;                         // frame tiles per 128-window tile (1 when B >= 128)
    int b_chunks;                    // ceil(B / 128)
    int MT, n_items;                 // 128-window tiles per channel, work items
    int padL, lead;
    int nsb, NS, NS_last;            // nsb - 1 sub-blocks of NS columns, the last of NS_last
    int Kspan;                       // K extent of one sub-block's MMA chain (multiple of 32)
    int a_kblocks;                   // 128-byte K blocks of A
    int a_kblocks_ld, last_w;        // K blocks that are loaded, and the bytes of the last of them (multiple of 16):
                                     // behind the last byte any output needs the band is zero, so whatever the
                                     // stage still holds there multiplies zeros (integers: no NaN can arise)
    int ksteps_last;                 // 32-byte K steps of the last (narrower) sub-block's MMA chain
    int b_rows;                      // rows of the band matrix = widest sub-block
    int band_chunks;                 // 16-byte chunks a band row can touch
    int a_bytes, b_bytes;            // per stage
    int staged;                      // outputs go through shared memory and TMA stores (else 16-byte global stores)
    int stage_w;                     // bytes per staged row of the wider epilogue warps (16 * ceil(chunks / EPI_PARTS))
    int box_rows;                    // utterances per TMA store box = min(32, rows_b)
    unsigned* status;
    QasrPrefetch next;               // constants of the kernel that follows
};

struct SharedTail {
    uint64_t full[2], empty[2], accfull[2], accempty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int build_ok[2];
    volatile int epi_go[2];          // per accumulator buffer: the polling epilogue warp saw it complete (0: it gave up)
    int8_t taps[2][128];
};

// which frame tile and which first utterance a 128-window tile covers
__device__ __forceinline__ void mtile_coords(const Params& p, int mt, int& tile0, int& b0) {
    if (p.b_chunks > 1) {
        tile0 = mt / p.b_chunks;
        b0 = (mt - tile0 * p.b_chunks) * 128;
    } else {
        tile0 = mt * p.tpm;
        b0 = 0;
    }
}

template <int MODE>
__device__ __forceinline__ int4 requant16_dw(const uint32_t (&r)[16], int mn, long long half64, int sn) {
    int q[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (MODE == 0) q[i] = ptx::mad_hi64((int)r[i], mn, half64);
        else if (MODE == 1) q[i] = ptx::mad_hi64((int)r[i], mn, half64) >> (sn - 32);
        else q[i] = (int)clamp_i8_ll(((long long)(int)r[i] * (long long)mn + half64) >> sn);
    }
    int4 out;
    out.x = (int)ptx::pack4_sat_s8(q[0], q[1], q[2], q[3]);
    out.y = (int)ptx::pack4_sat_s8(q[4], q[5], q[6], q[7]);
    out.z = (int)ptx::pack4_sat_s8(q[8], q[9], q[10], q[11]);
    out.w = (int)ptx::pack4_sat_s8(q[12], q[13], q[14], q[15]);
    return out;
}

__global__ void __launch_bounds__(THREADS, 1)
dw_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmXl,
             const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmYw, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* const A0 = smem;
    uint8_t* const A1 = A0 + p.a_bytes;
    uint8_t* const B0 = A1 + p.a_bytes;
    uint8_t* const B1 = B0 + p.b_bytes;
    uint32_t* const lines = reinterpret_cast<uint32_t*>(B1 + p.b_bytes);   // per group: 4 shifted tap lines
    uint8_t* const Ostage = reinterpret_cast<uint8_t*>(lines + 2 * 4 * LINE_WORDS);   // one block per epilogue warp
    SharedTail* sh = reinterpret_cast<SharedTail*>(Ostage + (p.staged ? EPI_WARPS * 32 * p.stage_w : 0));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // the band matrices start out zero; only their bands are ever rewritten
    for (int i = threadIdx.x; i < p.b_bytes / 16; i += THREADS) {
        reinterpret_cast<int4*>(B0)[i] = make_int4(0, 0, 0, 0);
        reinterpret_cast<int4*>(B1)[i] = make_int4(0, 0, 0, 0);
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[i]), BUILD_GROUP_WARPS + 1);   // builders + the TMA bytes
            ptx::mbar_init(ptx::smem_u32(&sh->empty[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->accfull[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->accempty[i]), EPI_GROUP_WARPS);
        }
        sh->abort_flag = 0;
        sh->build_ok[0] = sh->build_ok[1] = 1;
        ptx::mbar_fence_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* abort_flag = &sh->abort_flag;
    // The taps are constants of the layer, not results of the previous kernel, and their first touch comes
    // from DRAM: each builder thread holds the tap of its group's next item in a register, fetched one item
    // ahead; the first fetch is issued here, before the dependency wait.
    const int bgrp = warp / BUILD_GROUP_WARPS;
    const int btid = threadIdx.x - bgrp * BUILD_GROUP_THREADS;
    // The copies of one item are dealt over the group's warps first, then over lanes: the lanes of one warp
    // issue their copies one after the other (~140 cycles each), different warps side by side.
    const int bbox = (btid & 31) * BUILD_GROUP_WARPS + (btid >> 5);
    auto fetch_tap = [&](uint32_t n) -> int8_t {
        const long long it = (long long)blockIdx.x + (long long)n * gridDim.x;
        if (warp >= BUILD_WARPS || it >= p.n_items || btid >= p.K) return 0;
        return __ldg(p.w + (size_t)((int)it / p.MT) * p.K + btid);
    };
    int8_t tap_next = fetch_tap(bgrp);
    // coordinates of a builder group's item; those of the first one are ready before the dependency wait returns
    struct ItemAt { int c, tile0, b0, n_tiles, n_boxes, kb, ti; };
    auto locate = [&](uint32_t n) {
        ItemAt it;
        const long long item64 = (long long)blockIdx.x + (long long)n * gridDim.x;
        const int item = item64 < p.n_items ? (int)item64 : 0;
        it.c = item / p.MT;
        mtile_coords(p, item - it.c * p.MT, it.tile0, it.b0);
        it.n_tiles = min(p.tpm, p.tiles - it.tile0);
        it.n_boxes = it.n_tiles * p.a_kblocks_ld;
        it.kb = bbox / it.n_tiles;                 // the box this thread issues (if bbox < n_boxes)
        it.ti = bbox - it.kb * it.n_tiles;
        return it;
    };
    ItemAt at = locate(bgrp);
    if (threadIdx.x == 0) {   // kernel parameters: fetch them while the previous kernel drains
        ptx::tma_prefetch_desc(&tmX);
        ptx::tma_prefetch_desc(&tmXl);
        ptx::tma_prefetch_desc(&tmY);
        ptx::tma_prefetch_desc(&tmYw);
    }
    if (warp == MMA_WARP) prefetch_ranges_l2(p.next, lane);
    // everything above touched only this CTA's own state and constants; from here on the previous kernel's output is read
    ptx::grid_dep_launch();
    // The builders put the dependency wait off: taps, tap line and band of their first item depend only on the
    // layer's constants and are built while the previous kernel drains (that item's window loads are issued by
    // the epilogue warps, which do wait here); a builder waits before the first window load of its own.
    if (warp >= BUILD_WARPS) ptx::grid_dep_wait();

    if (warp < BUILD_WARPS) {
        // ------------------------------------------------------------------ builders
        // Two groups of four warps; group g owns stage g and builds every second item.
        const int grp = warp / BUILD_GROUP_WARPS;
        const int tid = threadIdx.x - grp * BUILD_GROUP_THREADS;
        uint8_t* const Astage = grp ? A1 : A0;
        uint8_t* const Bstage = grp ? B1 : B0;
        uint32_t* const line = lines + grp * 4 * LINE_WORDS;
        int8_t* const taps = sh->taps[grp];
        for (uint32_t n = grp;; n += 2, at = locate(n)) {
            const long long item64 = (long long)blockIdx.x + (long long)n * gridDim.x;
            if (item64 >= p.n_items) break;
            const int c = at.c, tile0 = at.tile0, b0 = at.b0, n_boxes = at.n_boxes;
            // A: one box [rows_b utterances][128 bytes] per frame tile and K block, each issued by its own
            // thread, dealt over the group's four warps (the host admits at most one box per builder thread);
            // frames outside [0, T) are filled with zeros by the copy engine
            auto load_windows = [&]() {
                if (bbox < n_boxes)
                    ptx::tma_load_3d(ptx::smem_u32(Astage + at.kb * A_KBLOCK_BYTES + at.ti * p.rows_b * 128),
                                     at.kb == p.a_kblocks_ld - 1 ? &tmXl : &tmX,
                                     (tile0 + at.ti) * p.NT * p.stride - p.padL + 128 * at.kb, c, b0, ptx::smem_u32(&sh->full[grp]));
            };
            const bool first_use = n == (uint32_t)grp;     // the stage has never been used: nothing to wait for
            // the first item's boxes are issued by the epilogue warps, which have nothing to do yet (one box per
            // warp side by side instead of three per builder warp one after the other); the bytes may land
            // before tid 0 announces them
            if (tid < p.K) taps[tid] = tap_next;
            tap_next = fetch_tap(n + 2);
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "n"(BUILD_GROUP_THREADS) : "memory");   // taps staged
            // The tap line belongs to the builders alone, so it is built before the stage is known to be free:
            // the wait for the MMAs that still read the stage's previous contents overlaps it.
            // tap line, four copies shifted by 0..3 bytes, 16 zero bytes in front
            for (int wi = tid; wi < 4 * LINE_WORDS; wi += BUILD_GROUP_THREADS) {
                const int r = wi / LINE_WORDS, idx = wi - r * LINE_WORDS;
                uint32_t word = 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int q = 4 * idx + e + r - 16;          // byte offset from the first tap
                    const int k = q >> (p.dil - 1);              // dilation is 1 or 2
                    if (q >= 0 && (k << (p.dil - 1)) == q && k < p.K) word |= (uint32_t)(uint8_t)taps[k] << (8 * e);
                }
                line[wi] = word;
            }
            if (tid == 0) {
                const bool ok = first_use || ptx::mbar_wait(ptx::smem_u32(&sh->empty[grp]), ((n >> 1) & 1u) ^ 1u, abort_flag, p.status);
                sh->build_ok[grp] = ok ? 1 : 0;
                if (ok) ptx::mbar_expect_tx(ptx::smem_u32(&sh->full[grp]),
                                            (uint32_t)(at.n_tiles * p.rows_b * (128 * (p.a_kblocks_ld - 1) + p.last_w)));
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "n"(BUILD_GROUP_THREADS) : "memory");   // tap line complete, go/no-go known
            if (!sh->build_ok[grp]) break;
            if (!first_use) {
                ptx::grid_dep_wait();       // returns at once after the first time
                load_windows();
            }
            // Bt band: row nn holds the taps starting at byte nn*stride + lead. K-major with the 128-byte
            // swizzle: 16-byte chunk kc of row nn lives in K block kc / 8 at row nn, chunk (kc % 8) ^ (nn % 8).
            {
                const int span = (p.K - 1) * p.dil;
                const uint32_t kblock_bytes = (uint32_t)p.b_rows * 128u;
                for (int nn = tid; nn < p.b_rows; nn += BUILD_GROUP_THREADS) {
                    const int first = nn * p.stride + p.lead;
                    int kc = first >> 4;
                    int o = 16 - (first & 15);                                 // offset into the tap line, >= 1
                    uint8_t* const rowp = Bstage + nn * 128;
                    for (; 16 * kc <= first + span; ++kc, o += 16) {
                        const uint32_t* src = line + (o & 3) * LINE_WORDS + (o >> 2);
                        int4 v;
                        v.x = (int)src[0]; v.y = (int)src[1]; v.z = (int)src[2]; v.w = (int)src[3];
                        *reinterpret_cast<int4*>(rowp + (uint32_t)(kc >> 3) * kblock_bytes + (((kc & 7) ^ (nn & 7)) << 4)) = v;
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->full[grp]));
            // taps and tap line are rewritten at the top of the next item: every builder must be done with them
            asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "n"(BUILD_GROUP_THREADS) : "memory");
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------------ MMA issuer
        // the whole warp walks the loop (all lanes poll the barriers); one elected lane issues
        {
            // A single thread issues every MMA, so the loop carries the descriptors as running values: only
            // their start-address field (bits 0..13, 16-byte units) changes from one MMA to the next.
            const uint32_t idesc_mid = ptx::idesc_i8(128, p.NS, 0, 0);
            const uint32_t idesc_last = ptx::idesc_i8(128, p.NS_last, 0, 0);
            // A and Bt: K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart; the next
            // K block is 16 KiB further in A (128 windows) and b_rows * 128 bytes further in Bt. A 32-byte
            // K step never straddles a block (sub-blocks start on multiples of 32 bytes).
            const uint64_t a_d0 = ptx::smem_desc(ptx::smem_u32(A0), 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t a_d1 = ptx::smem_desc(ptx::smem_u32(A1), 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t b_d0 = ptx::smem_desc(ptx::smem_u32(B0), 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t b_d1 = ptx::smem_desc(ptx::smem_u32(B1), 16, 1024, ptx::SWIZZLE_128B);
            const uint32_t b_wrap = (uint32_t)p.b_rows * 8u - 8u;   // 16-byte units from the end of a row to the next K block
            const int ksteps = p.Kspan >> 5, nsb = p.nsb, NS = p.NS;
            const int sb_koff = NS * p.stride;                       // bytes of K between sub-blocks (multiple of 32)
            const uint32_t full0 = ptx::smem_u32(&sh->full[0]), empty0 = ptx::smem_u32(&sh->empty[0]);
            const uint32_t accfull0 = ptx::smem_u32(&sh->accfull[0]), accempty0 = ptx::smem_u32(&sh->accempty[0]);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                ok = ptx::mbar_try(full0 + s * 8, ph) || ptx::mbar_wait(full0 + s * 8, ph, abort_flag, p.status);
                ok = ok && (ptx::mbar_try(accempty0 + s * 8, ph ^ 1u) || ptx::mbar_wait(accempty0 + s * 8, ph ^ 1u, abort_flag, p.status));
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint64_t a_stage = s ? a_d1 : a_d0;
                const uint64_t b_stage = s ? b_d1 : b_d0;
                const uint32_t d_tmem = tmem_base + s * ACC_STRIDE;
                int koff = 0;
                if (ptx::elect_one()) {
                for (int sb = 0; sb < nsb; ++sb) {
                    const uint32_t idesc = sb == nsb - 1 ? idesc_last : idesc_mid;
                    const int ks = sb == nsb - 1 ? p.ksteps_last : ksteps;
                    uint32_t within = (uint32_t)koff & 127u;
                    uint64_t ad = a_stage + (((uint32_t)koff >> 7) << 10) + (within >> 4);
                    uint64_t bd = b_stage;
                    uint32_t b_within = 0;
                    uint32_t accumulate = 0;
                    for (int j = 0; j < ks; ++j) {
                        ptx::mma_i8(d_tmem + sb * NS, ad, bd, idesc, accumulate);
                        accumulate = 1;
                        ad += 2;
                        within += 32;
                        if (within == 128) { within = 0; ad += 1024 - 8; }   // on to the next 16 KiB K block
                        bd += 2;
                        b_within += 32;
                        if (b_within == 128) { b_within = 0; bd += b_wrap; }
                    }
                    koff += sb_koff;
                }
                ptx::tc_commit(empty0 + s * 8);
                ptx::tc_commit(accfull0 + s * 8);
                }
                __syncwarp();
                s ^= 1u;
                if (s == 0) ph ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;
        const int egrp = (warp - BUILD_WARPS) / EPI_GROUP_WARPS;       // which accumulator buffer / every second item
        const int part = ((warp - BUILD_WARPS) >> 2) % EPI_PARTS;
        const int n_chunks = p.NT >> 4;
        const int c_lo = part * n_chunks / EPI_PARTS;
        const int c_hi = (part + 1) * n_chunks / EPI_PARTS;
        const int row = quarter * 32 + lane;
        const int ti = row / p.rows_b;                 // frame tile within the 128-window tile
        const int rb = row - ti * p.rows_b;            // utterance within the box
        // Staged form: a warp's 32 windows are 32 / box_rows runs of box_rows consecutive utterances of one
        // frame tile; it stages its [32 windows][16 * (c_hi - c_lo) frames] block and lanes 0 .. 32 / box_rows - 1
        // each write one run with a TMA store (box: frames x 1 channel x box_rows utterances), which also clips
        // frames >= T_out and utterances >= B. Thirty-two 16-byte global stores to 32 different rows per warp
        // instruction were what bounded this kernel; the stores of one warp now cost four shared-memory wavefronts.
        const int my_w = 16 * (c_hi - c_lo);
        const CUtensorMap* const my_map = my_w == p.stage_w ? &tmYw : &tmY;
        uint8_t* const Ow = Ostage + (warp - BUILD_WARPS) * 32 * p.stage_w;
        const int srow = quarter * 32 + lane * p.box_rows;       // first window of the run this lane stores
        const int sti = srow / p.rows_b;
        const int srb = srow - sti * p.rows_b;
        const bool storer = p.staged && my_w > 0 && lane * p.box_rows < 32;
        {
            // window loads of the two builder groups' first items: box j of group g by epilogue thread
            // (warp j % EPI_WARPS, lane j / EPI_WARPS) counting over both groups
            const int ew = warp - BUILD_WARPS;
            for (int g = 0; g < 2; ++g) {
                const long long it64 = (long long)blockIdx.x + (long long)g * gridDim.x;
                if (it64 >= p.n_items) break;
                const int item = (int)it64;
                const int c0 = item / p.MT;
                int tile0, b0;
                mtile_coords(p, item - c0 * p.MT, tile0, b0);
                const int n_tiles = min(p.tpm, p.tiles - tile0);
                const int n_boxes = n_tiles * p.a_kblocks_ld;
                uint8_t* const Astage = g ? A1 : A0;
                for (int j = lane * EPI_WARPS + ew; j < n_boxes; j += 32 * EPI_WARPS) {
                    const int kb = j / n_tiles, ti = j - kb * n_tiles;
                    ptx::tma_load_3d(ptx::smem_u32(Astage + kb * A_KBLOCK_BYTES + ti * p.rows_b * 128),
                                     kb == p.a_kblocks_ld - 1 ? &tmXl : &tmX,
                                     (tile0 + ti) * p.NT * p.stride - p.padL + 128 * kb, c0, b0, ptx::smem_u32(&sh->full[g]));
                }
            }
        }
        uint32_t n = (uint32_t)egrp;
        bool ok = true;
        // the requantisation constants of this group's next item are fetched while this one is requantised
        const long long first = (long long)blockIdx.x + (long long)egrp * gridDim.x;
        const long long step = (long long)EPI_GROUPS * gridDim.x;
        int m_next = 0, sft_next = 1;
        if (first < p.n_items) load_rq(p.mult, p.shift, (int)first / p.MT, m_next, sft_next, p.status);
        for (long long item64 = first; item64 < p.n_items && ok; item64 += step, n += EPI_GROUPS) {
            const int item = (int)item64;
            const int c = item / p.MT, mt = item - c * p.MT;
            const int s = n & 1u;                     // == egrp
            const int m = m_next, sft = sft_next;
            if (item64 + step < p.n_items) load_rq(p.mult, p.shift, (int)(item64 + step) / p.MT, m_next, sft_next, p.status);
            const int kmax = min(__clz(m) - 1, 62 - sft);
            const int k = (sft <= 32 && 32 - sft <= kmax) ? 32 - sft : kmax;   // same dyadic number, shift 32 if possible
            const int mn = m << k, sn = sft + k;
            const long long half64 = 1LL << (sn - 1);
            const int mode = sn == 32 ? 0 : (sn > 32 ? 1 : 2);      // uniform: one channel per item
            int tile0, b0;
            mtile_coords(p, mt, tile0, b0);
            const int i = tile0 + ti;
            const int b = b0 + rb;
            const bool valid = ti < p.tpm && i < p.tiles && b < p.B;
            const int valid_len = valid ? min(p.NT, p.T_out - i * p.NT) : 0;
            int8_t* yrow = p.y + ((size_t)(valid ? b : 0) * p.C + c) * p.T_out + (size_t)(valid ? i : 0) * p.NT;
            // One warp of the group polls the barrier; the others sleep in a hardware barrier until it has seen the
            // accumulator (waiting warps then take no issue slots). The polling warp always arrives (its wait is
            // bounded) and passes its verdict on through shared memory.
            if (warp == BUILD_WARPS + egrp * EPI_GROUP_WARPS) {
                const bool seen = ptx::mbar_wait(ptx::smem_u32(&sh->accfull[s]), (n >> 1) & 1u, abort_flag, p.status);
                if (lane == 0) sh->epi_go[s] = seen ? 1 : 0;
            }
            asm volatile("bar.sync %0, %1;" ::"r"(3 + egrp), "n"(32 * EPI_GROUP_WARPS) : "memory");
            ok = sh->epi_go[s] != 0;
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + s * ACC_STRIDE;
            if (p.staged) {     // this warp's previous stores must have finished reading its staging block
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
            }
            uint8_t* const orow = Ow + lane * my_w - c_lo * 16;     // chunk ch lands at orow + 16 * ch
            for (int ch = c_lo; ch < c_hi; ++ch) {
                uint32_t acc[16];
                __syncwarp();
                ptx::tmem_ld16(taddr + ch * 16, acc);
                ptx::tmem_ld_wait(acc);
                int4 out;
                if (mode == 0) out = requant16_dw<0>(acc, mn, half64, sn);
                else if (mode == 1) out = requant16_dw<1>(acc, mn, half64, sn);
                else out = requant16_dw<2>(acc, mn, half64, sn);
                if (p.staged) *reinterpret_cast<int4*>(orow + ch * 16) = out;
                else if (16 * ch < valid_len) *reinterpret_cast<int4*>(yrow + ch * 16) = out;   // 16 frames: all or nothing
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->accempty[s]));
            if (p.staged) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                const int si = tile0 + sti;
                if (storer && sti < p.tpm && si < p.tiles && b0 + srb < p.B) {
                    asm volatile(
                        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                        ::"l"(my_map), "r"(si * p.NT + c_lo * 16), "r"(c), "r"(b0 + srb),
                          "r"(ptx::smem_u32(Ow + lane * p.box_rows * my_w))
                        : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        // the staging blocks must outlive the stores' reads of them; the writes themselves complete with the grid
        if (p.staged) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
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
    if (warp == MMA_WARP) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace dwtc
}  // namespace qasr

int qasr_dw_tc_init(qasr_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(qasr::dwtc::dw_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "cudaFuncSetAttribute(dw_tc_kernel) failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return QASR_OK;
}

// Returns 1 if enqueued, 0 if the shape is not one this kernel takes, negative on error.
int qasr_launch_dw_tc(qasr_ctx* ctx, const QasrDwArgs& a) {
    using namespace qasr::dwtc;
    if (a.T % 16 != 0 || a.T_out % 16 != 0) return 0;
    if (((uintptr_t)a.x & 15u) || ((uintptr_t)a.y & 15u)) return 0;
    if ((a.K - 1) * a.dilation + 1 + 32 > 4 * LINE_WORDS - 16) return 0;
    // the boxes of several frame tiles are stacked in one swizzled K block: keep every box a whole
    // number of 8-row swizzle groups
    if (a.B < 128 && a.B % 8 != 0) return 0;
    Params p;
    memset(&p, 0, sizeof(p));
    p.w = a.w; p.mult = a.mult; p.shift = a.shift; p.y = a.y;
    p.B = a.B; p.C = a.C; p.T = a.T; p.T_out = a.T_out; p.K = a.K; p.stride = a.stride; p.dil = a.dilation;
    const int pad = a.dilation * (a.K - 1) / 2;
    p.padL = (pad + 15) & ~15;
    p.lead = p.padL - pad;
    p.rows_b = a.B < 128 ? a.B : 128;
    p.b_chunks = (a.B + 127) / 128;
    p.tpm = a.B < 128 ? 128 / a.B : 1;
    // frame tile: cheapest by a rough count of cycles per SM (windows come in groups of 128)
    double best = 1e30;
    for (int tiles = (a.T_out + 255) / 256; tiles <= a.T_out / 16; ++tiles) {
        const int nt = ((a.T_out + tiles - 1) / tiles + 15) & ~15;
        if ((a.T_out + nt - 1) / nt != tiles) continue;
        const long long mt = p.b_chunks > 1 ? (long long)tiles * p.b_chunks : (tiles + p.tpm - 1) / p.tpm;
        const int nsb = nt < 128 ? 1 : (nt / 64 > MAX_SB ? MAX_SB : nt / 64);
        const int ns_last = nt - 64 * (nsb - 1);
        const int span = ns_last * a.stride + (a.K - 1) * a.dilation + 32;    // K extent of a sub-block, roughly
        const int kga = nt * a.stride + (a.K - 1) * a.dilation + 48;          // bytes loaded per window
        const double cost = (double)mt * (128.0 * nt * span / 8192.0 + 0.5 * kga + 400.0);
        if (cost < best) { best = cost; p.NT = nt; p.tiles = tiles; }
    }
    if (ctx->force_dw_nt >= 16 && ctx->force_dw_nt <= 256 && ctx->force_dw_nt % 16 == 0 && ctx->force_dw_nt <= ((a.T_out + 15) & ~15)) {
        p.NT = ctx->force_dw_nt;                  // tuning aid: the caller's frame tile instead of the cost model's
        p.tiles = (a.T_out + p.NT - 1) / p.NT;
    }
    if (!p.NT) return 0;
    p.MT = p.b_chunks > 1 ? p.tiles * p.b_chunks : (p.tiles + p.tpm - 1) / p.tpm;
    if ((long long)a.C * p.MT > 0x7fffffffLL) return 0;
    p.n_items = a.C * p.MT;
    // Output staging: possible when a warp's 32 windows split into whole runs of utterances of one frame tile
    {
        const int n_chunks = p.NT / 16;
        p.stage_w = 16 * ((n_chunks + EPI_PARTS - 1) / EPI_PARTS);
        p.box_rows = p.rows_b < 32 ? p.rows_b : 32;
        p.staged = (p.rows_b % 32 == 0 || 32 % p.rows_b == 0) ? 1 : 0;
    }
    // Sub-blocks of the MMA N dimension share one band matrix: 128 columns when the two stages then still
    // fit in shared memory (fewer, larger MMAs: the single issuing thread is the scarce resource), else 64.
    // Where the staging blocks do not fit beside the two stages, the outputs go out as 16-byte global stores.
    size_t smem = 0;
    const int may_stage = p.staged;
    for (int attempt = 0; attempt < 4 && !smem; ++attempt) {
        const int unit = attempt < 2 ? 128 : 64;
        p.staged = (attempt & 1) ? 0 : may_stage;
        if ((attempt & 1) && !may_stage) continue;      // same as the attempt before
        p.nsb = (p.NT + unit - 1) / unit;
        if (p.nsb > MAX_SB) continue;
        p.NS = p.nsb == 1 ? p.NT : unit;
        p.NS_last = p.NT - unit * (p.nsb - 1);
        if (p.NS_last > 256) return 0;
        p.b_rows = p.NS_last > p.NS ? p.NS_last : p.NS;
        p.Kspan = ((p.b_rows - 1) * a.stride + p.lead + (a.K - 1) * a.dilation + 1 + 31) & ~31;
        const int kga = (p.nsb - 1) * p.NS * a.stride + p.Kspan;
        p.a_kblocks = (kga + 127) / 128;
        p.band_chunks = ((a.K - 1) * a.dilation + 15) / 16 + 1;
        {
            // the last input byte any output of a window needs, and the K extent of the last sub-block's chain
            const int need = (p.NT - 1) * a.stride + p.lead + (a.K - 1) * a.dilation + 1;
            p.a_kblocks_ld = (need + 127) / 128;
            p.last_w = ((need - 128 * (p.a_kblocks_ld - 1)) + 15) & ~15;
            const int span_last = (p.NS_last - 1) * a.stride + p.lead + (a.K - 1) * a.dilation + 1;
            p.ksteps_last = (span_last + 31) / 32;
            if (p.ksteps_last > p.Kspan / 32) p.ksteps_last = p.Kspan / 32;
        }
        p.a_bytes = p.a_kblocks * A_KBLOCK_BYTES;
        p.b_bytes = ((p.Kspan + 127) / 128) * p.b_rows * 128;     // whole 128-byte K blocks of the swizzled band
        smem = 1024 + 2 * (size_t)(p.a_bytes + p.b_bytes) + 2 * 4 * LINE_WORDS * 4 + sizeof(SharedTail) +
               (p.staged ? (size_t)EPI_WARPS * 32 * p.stage_w : 0);
        if (smem > 227 * 1024 || p.tpm * p.a_kblocks > BUILD_GROUP_THREADS) smem = 0;
    }
    if (!smem) return 0;
    p.status = ctx->d_status;
    p.next = ctx->prefetch;
    memset(&ctx->prefetch, 0, sizeof(ctx->prefetch));

    CUtensorMap tmX, tmXl;
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.T, (cuuint64_t)a.C, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.T, (cuuint64_t)a.T * a.C};
        cuuint32_t box[3] = {128u, 1u, (cuuint32_t)p.rows_b};
        if (!qasr_encode_map_u8(ctx, &tmX, a.x, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
        // the last loaded K block: only as wide as the outputs need it (same 128-byte row pitch and swizzle)
        box[0] = (cuuint32_t)p.last_w;
        if (!qasr_encode_map_u8(ctx, &tmXl, a.x, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B)) return QASR_ERR_CUDA;
    }
    CUtensorMap tmY = tmX, tmYw = tmX;     // unused without staging
    if (p.staged) {
        cuuint64_t dims[3] = {(cuuint64_t)a.T_out, (cuuint64_t)a.C, (cuuint64_t)a.B};
        cuuint64_t strides[2] = {(cuuint64_t)a.T_out, (cuuint64_t)a.T_out * a.C};
        cuuint32_t box[3] = {(cuuint32_t)p.stage_w, 1u, (cuuint32_t)p.box_rows};
        if (!qasr_encode_map_u8(ctx, &tmYw, a.y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
        const int narrow = 16 * ((p.NT / 16) / EPI_PARTS);
        box[0] = (cuuint32_t)(narrow > 0 ? narrow : p.stage_w);
        if (!qasr_encode_map_u8(ctx, &tmY, a.y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return QASR_ERR_CUDA;
    }
    const int grid = p.n_items < qasr_grid_slots(ctx) ? p.n_items : qasr_grid_slots(ctx);
    QasrLaunchScope ls(ctx, QASR_K_DW_TC, qasr_dw_macs(a), qasr_dw_bytes(a));
    cudaError_t e = qasr_launch_overlapped(ctx, dw_tc_kernel, dim3(grid), dim3(THREADS), smem, tmX, tmXl, tmY, tmYw, p);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "dw_tc_kernel launch failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return 1;
}
