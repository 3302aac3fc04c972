// Weight-gradient pass on the 5th-generation tensor cores (stride-1 layers).
//
//   dw[k, r, s, c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p+r-pad_h, q+s-pad_w, c]
//
// GEMM view per tap (r, s): M = K output maps, N = C input maps, reduction over
// the N*P*Q output pixels.  The reduction index is the OUTER dimension of both
// NHWC tensors, so both operands are "MN-major": a TMA box {32 maps, 32 pixels}
// lands in shared memory as 32 rows (one per pixel) of 128 bytes, swizzled in
// 32-byte chunks, which is the MN-major operand layout tcgen05.mma takes for
// 32-bit elements.  The x box is the dy box shifted by the tap, with zero
// padding supplied by TMA's out-of-bounds fill.
//
// Columns of the MMA are organised in "runs": a run is L consecutive 32-map
// groups of x for one tap (L <= 8), fetched by one TMA instruction through a
// 5-D view {32 maps, w, h, n, group} of the tensor.  A CTA accumulates up to 8
// groups (N <= 256) = several runs, which may belong to different taps: layers
// with few input maps (C = 64: 2 groups per tap) then still fill a 128 x 192 or
// 128 x 256 tile and read dy once for 3-4 taps instead of once per tap.
//
// The output is tiny compared with the reduction (Sec. 2.4/2.5 make the same
// observation), so the pixel range is split across CTAs ("privatise and
// reduce"): a work item is (128-row k tile, block of runs, pixel split); each CTA
// accumulates its item in TMEM and either writes a partial tile to the
// workspace (second pass adds the splits in a fixed order) or adds it to dw with
// fp32 atomics.
//
// Haloed x ("xhalo", single-CTA items of stride-1 layers with S > 1 and few input maps): the S taps of one kernel
// row read pixel boxes that overlap in all but S-1 columns, so ONE box of (bw + S - 1) x bh x bn pixels per 32-map
// group is fetched per k-step and every tap is a view of it shifted by one 128-byte row: an MMA takes the S taps of
// one map group as S consecutive 32-column groups 128 bytes apart (the descriptor's leading-dimension offset),
// i.e. N = 32*S columns, one MMA per map group and 8 pixels.  A work item is then (k tile, kernel row, pixel
// split).  For C = 64, 3x3 this cuts the bytes fetched per 64 pixels from 80 to 50 KB; such layers sit at the
// L2-to-SM ceiling, not at the tensor pipe's.
//
// Pooled dy ("dy_pool" launches, for a layer whose output went through a 2x2 max pool and that has no
// backward-data pass of its own, i.e. the first layer): dy is never materialised.  The eight epilogue warps, idle
// during the main loop, build each k-step's dy tile in shared memory themselves from the pooled gradient and the
// windows' position codes (one (pooled pixel, 4 maps) item per thread: the gradient goes to the coded position of
// the window, zeros to the other three, everything rounded to TF32 as a TMA load would), in exactly the layout a
// TMA load of dy produces (rows of 128 bytes per pixel and 32-map group, 32-byte chunks XOR-ed with row & 3), and
// arrive on the slot's barrier next to the x copy.  They also sum what they scatter: the bias gradient.
//
// A k-step is one pixel box of 32 or 64 pixels (4 or 8 MMAs of 8 pixels).  With an
// even number of k tiles, two CTAs of a cluster take k tiles 2i and 2i+1 of the
// same run block and pixel split: each loads its own dy tile and half of the x
// runs, and the even CTA issues M = 256 MMAs for both (cta_group::2).
#include <stdlib.h>

#include <mutex>
#include <string>
#include <type_traits>
#include <unordered_map>

#include "pcl_internal.h"
#include "pcl_ptx.cuh"

namespace pcl {

namespace {

constexpr int kMaxStages = 8;
constexpr int kWgradThreads = 352;     // warp 0 producer, warps 1 and 10 MMA issuers, warps 2-9 epilogue (two per TMEM lane quarter)
constexpr int kSecondIssuerWarp = 10;
constexpr int kWgradThreadsWide = 608; // pooled-dy launches with two issuers: warps 11-18 are a second group of dy builders
constexpr int kSmemBudget = 224 * 1024;
constexpr int kExpanderWarps = 8;      // the epilogue warps, which build the dy tiles of pooled-dy launches during the main loop

struct WgradParams {
    int bw_log2, bh_log2;     // pixel box bw x bh x (pix/(bw*bh))
    int pix;                  // pixels (reduction indices) per k-step: 32 or 64
    int boxes_q, boxes_p, boxes_n;
    int k_tiles;
    int L;                    // 32-map groups per run
    int runs_per_tap;         // ceil(C/32) / L
    int total_runs;           // R*S*runs_per_tap
    int rpi;                  // runs per work item (rpi*L <= 8); even in pair mode
    int run_blocks;           // ceil(total_runs / rpi)
    int R, S, pad_h, pad_w;
    int stride_h, stride_w, dil_w;   // convolution strides; pixels between consecutive taps of a kernel row
    int K, C;
    int splits, boxes_per_split;
    int stages, tmem_cols;
    int KS;                   // k-steps per pipeline slot; > 1 for narrow column blocks
    int use_atomics;
    int grouped;              // x: 5-D tensor map (one TMA instruction per run) or 4-D per-group boxes (L == 1)
    int grouped_dy;           // dy: 5-D tensor map (all four 32-map groups in one instruction)
    int x_taprows;            // x: 5-D map whose 5th dimension is the tap row (few-channel path): one instruction per k-step
    int xhalo;                // haloed x boxes: item = (k tile, kernel row, split), one x copy per k-step (see the header)
    int cg;                   // xhalo: 32-map groups of x (C / 32)
    int x_group_bytes;        // xhalo: bytes of one group's haloed box, (bw + S - 1) * bh * bn * 128
    int x_step_bytes;         // xhalo: bytes of a k-step (dy tile + cg haloed boxes, rounded up to 1 KB)
    // pooled dy (see the header): dy_pool [N][P/2][Q/2][K], codes the same shape in bytes (bits 0-1 position in the
    // window, bit 2 "maximum <= 0"); relu_mask: windows with bit 2 set contribute nothing; db_rows [splits * 8][K]
    const float* dy_pool;
    const unsigned char* codes;
    int relu_mask;
    float* db_rows;
    int N, P, Q;              // output size (for the pooled tile's bounds)
    float* out;               // dw, or the partial-sum workspace [splits][K*R*S*C]
    size_t split_stride;      // K*R*S*C (0 when writing straight to dw)
    // duo: two issuing threads take the pipeline slots alternately (the number of slots is even, so a slot always
    // belongs to the same thread), each into an accumulator of its own, acc_cols columns apart; the epilogue adds
    // the two in a fixed order.  What bounds a single-CTA item is the issuing thread (~100-140 cycles per MMA,
    // whatever its width), not the tensor pipe.
    int sgd;                  // unsplit launch: the epilogue writes out[i] - lr * (the tile) instead of the tile (out = the weights)
    float lr;
    int duo, acc_cols;
    int dy_groups;            // 32-map groups of a k-step's dy tile (4, fewer for pooled dy with K < 128)
    int inject_short_copy;    // test mode: the first slot is armed for 16 bytes more than are copied (see the forward kernel)
    unsigned int* status;     // device status word (status[1]: limit of the bounded waits in microseconds)
};

// One box row of a haloed-x k-step: kSteps MMA steps of 8 pixels, each one MMA per map group (kCg of them) over the
// S taps.  Straight-line: every instruction of the issuing role costs cycles of the k-step budget.
template <int kSteps, int kCg>
__device__ __forceinline__ void xhalo_row(uint32_t d_tmem, uint32_t xn, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                          uint32_t idesc, uint32_t acc_first, uint32_t xg16) {
#pragma unroll
    for (int m = 0; m < kSteps; ++m)
#pragma unroll
        for (int g = 0; g < kCg; ++g)
            umma_tf32(d_tmem + g * xn, (uint64_t(hi) << 32) | (a_lo + 64u * m), (uint64_t(hi) << 32) | (b_lo + 64u * m + g * xg16),
                      idesc, m == 0 ? acc_first : 1u);
}

// kPair: see the header.  Pair mode needs grouped x and dy maps; every item then has rpi runs (runs past the
// last tap read zeros through the out-of-bounds fill and are not stored).
// kWide (pooled dy with two issuers): sixteen warps build the dy tiles, in two groups that take the pipeline slots
// alternately like the issuing threads do -- a builder warp is a chain of dependent instructions per k-step, and two
// warps per scheduler cannot hide it.
// kSgd: the epilogue of an unsplit launch applies the SGD update in place (an instantiation of its own: the prefetched old
// weights would cost the plain epilogue registers and a branch per chunk).
template <bool kPair, bool kWide = false, bool kSgd = false>
__global__ void __launch_bounds__(kWide ? kWgradThreadsWide : kWgradThreads, 1)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap tmDy, const __grid_constant__ CUtensorMap tmX, WgradParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages];
    __shared__ uint64_t empty_bar[kMaxStages];
    __shared__ uint64_t tmem_full_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t pair_rank = kPair ? cluster_ctarank() : 0u;

    // work item of this CTA (pair: of this cluster; the two CTAs take k tiles 2i and 2i + 1)
    int item = kPair ? int(cluster_id_x()) : int(blockIdx.x);
    const int split = item % p.splits;   item /= p.splits;
    const int rb = item % p.run_blocks;
    const int kt = kPair ? 2 * (item / p.run_blocks) + int(pair_rank) : item / p.run_blocks;
    const int run0 = rb * p.rpi;
    const int nruns = kPair ? p.rpi : ((run0 + p.rpi <= p.total_runs) ? p.rpi : p.total_runs - run0);
    const int n_groups = p.xhalo ? p.cg * p.S : nruns * p.L;      // 32-column groups of this item's accumulator
    const int my_runs = kPair ? nruns >> 1 : nruns;   // runs this CTA loads (pair: its half of the columns)
    const int my_run0 = run0 + int(pair_rank) * my_runs;
    const uint32_t group_bytes = p.pix * 128;         // one {32 maps x pix pixels} box
    // 128 output maps; pooled-dy launches of layers with K < 128 build only the groups that exist, and the MMAs' rows
    // beyond them read the x tile behind (finite numbers into accumulator rows that are never stored; the slot
    // holds at least four groups, so the operand stays inside it)
    const uint32_t a_bytes = p.dy_groups * group_bytes;
    const uint32_t step_bytes = p.xhalo ? uint32_t(p.x_step_bytes)
                                        : a_bytes + (kPair ? (p.rpi >> 1) : p.rpi) * p.L * group_bytes;   // one k-step (same for every item)
    const uint32_t stage_bytes = p.KS * step_bytes;                     // a slot holds KS k-steps
    const uint32_t tx_bytes = (p.dy_pool ? 0u : a_bytes) + (p.xhalo ? uint32_t(p.cg) * p.x_group_bytes : my_runs * p.L * group_bytes);   // (pooled dy: written by the epilogue warps)

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full_bar[s], p.dy_pool ? 1 + kExpanderWarps : 1);     // + one arrival per warp that builds dy
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&tmem_full_bar, p.duo ? 2 : 1);
        abort_flag = 0;
        mbar_fence_init();
        prefetch_tmap(&tmDy);
        prefetch_tmap(&tmX);
    }
    if (warp == 1) {
        if constexpr (kPair) { tmem_alloc_pair(&tmem_base_slot, p.tmem_cols); tmem_relinquish_pair(); }
        else { tmem_alloc(&tmem_base_slot, p.tmem_cols); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync_all();     // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    const int total_boxes = p.boxes_q * p.boxes_p * p.boxes_n;
    const int box_begin = split * p.boxes_per_split;
    int box_end = box_begin + p.boxes_per_split;
    if (box_end > total_boxes) box_end = total_boxes;
    const int kiters = box_end > box_begin ? box_end - box_begin : 0;
    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2, bn = p.pix >> (p.bw_log2 + p.bh_log2);

    if (warp == 0) {
        // The whole warp runs the loop and an elected lane issues the copies; the loop is kept to a few instructions
        // per copy: addresses advance by addition, run coordinates are decoded once.
        {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            int run_dw[8], run_dh[8], run_c[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int run = my_run0 + (j < my_runs ? j : 0);
                if (run < p.total_runs) {
                    const int tap = run / p.runs_per_tap;
                    const int cg0 = (run - tap * p.runs_per_tap) * p.L;
                    const int r = tap / p.S, s = tap - r * p.S;
                    run_dw[j] = s * p.dil_w - p.pad_w;
                    run_dh[j] = r - p.pad_h;
                    run_c[j] = p.grouped ? cg0 : cg0 * 32;
                } else {
                    // (pair mode only) a run past the last tap: a group coordinate outside the tensor reads zeros
                    run_dw[j] = 0; run_dh[j] = 0; run_c[j] = (p.C + 31) / 32;
                }
            }
            int qi = box_begin % p.boxes_q;
            int pi = (box_begin / p.boxes_q) % p.boxes_p;
            int ni = box_begin / (p.boxes_q * p.boxes_p);
            const uint32_t run_bytes = p.L * group_bytes;
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]), ring0 = smem_u32(smem);
            const uint32_t full_dst0 = kPair ? map_to_cta(&full_bar[0], 0) : full0;     // where the copies complete
            uint32_t full_a = full0, empty_a = empty0, full_dst = full_dst0, slot_a = ring0;
            uint32_t dst = ring0;
            int sub = 0;                                         // position of the k-step inside its slot
            int q0 = qi * bw, p0 = pi * bh, n0 = ni * bn;
            const int xsw = p.stride_w, xsh = p.stride_h;      // x coordinates of a box: the dy box's times the stride
            for (int b = box_begin; b < box_end; ++b) {
                if (sub == 0) {
                    if (!bounded_wait_addr_warp(empty_a, phase ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) { ok = false; break; }
                    const int nst = box_end - b < p.KS ? box_end - b : p.KS;
                    // pair: both CTAs' copies complete on the leader's barrier, which its producer arms
                    if (!kPair) mbar_expect_tx_addr(full_a, nst * tx_bytes + (p.inject_short_copy && issued == 0 ? 16 : 0));
                    else if (pair_rank == 0) mbar_expect_tx_addr(full_a, 2 * nst * tx_bytes);
                    dst = slot_a;
                }
                if (p.dy_pool) {
                    // (no dy copy: the epilogue warps write the tile)
                } else if (p.grouped_dy) {
                    tma_load_5d_addr<kPair>(dst, &tmDy, full_dst, 0, q0, p0, n0, kt * 4);
                } else {
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        tma_load_4d_addr<kPair>(dst + g * group_bytes, &tmDy, full_dst, kt * 128 + g * 32, q0, p0, n0);
                }
                const uint32_t xdst = dst + a_bytes;
                if (p.xhalo) {
                    // all map groups of the haloed box of kernel row `rb` (columns q0 - pad_w .. q0 + bw + S - 2 - pad_w)
                    tma_load_5d_addr<kPair>(xdst, &tmX, full_dst, 0, q0 - p.pad_w, p0 + rb - p.pad_h, n0, 0);
                } else if (p.x_taprows) {
                    tma_load_5d_addr<kPair>(xdst, &tmX, full_dst, 0, q0 + run_dw[0], p0 + run_dh[0], n0, 0);
                } else if (p.grouped) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < my_runs)
                            tma_load_5d_addr<kPair>(xdst + j * run_bytes, &tmX, full_dst, 0, q0 * xsw + run_dw[j],
                                                    p0 * xsh + run_dh[j], n0, run_c[j]);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < my_runs)
                            tma_load_4d_addr<kPair>(xdst + j * run_bytes, &tmX, full_dst, run_c[j], q0 * xsw + run_dw[j],
                                                    p0 * xsh + run_dh[j], n0);
                }
                // next pixel box
                q0 += bw;
                if (++qi == p.boxes_q) {
                    qi = 0; q0 = 0; p0 += bh;
                    if (++pi == p.boxes_p) { pi = 0; p0 = 0; n0 += bn; }
                }
                dst += step_bytes;
                if (++sub == p.KS || b == box_end - 1) {
                    sub = 0;
                    ++issued;
                    full_a += 8; empty_a += 8; full_dst += 8; slot_a += stage_bytes;
                    if (++stage == p.stages) {
                        stage = 0; phase ^= 1u;
                        full_a = full0; empty_a = empty0; full_dst = full_dst0; slot_a = ring0;
                    }
                }
            }
            if (!ok) {
                // Gave up: copies already issued still land in this CTA's shared memory; wait (bounded) for them.
                const int pending = issued < p.stages ? issued : p.stages;
                for (int j = 0; j < pending; ++j) {
                    if (--stage < 0) { stage = p.stages - 1; phase ^= 1u; }
                    for (uint32_t spin = 0; spin < (1u << 20); ++spin)
                        if (mbar_try_wait(&full_bar[stage], phase)) break;
                }
            }
        }
    } else if (warp == 1 || warp == kSecondIssuerWarp) {
        const uint32_t issuer = warp == 1 ? 0u : 1u;
        const uint32_t nis = p.duo ? 2u : 1u;
        if (pair_rank == 0 && issuer < nis) {     // the whole warp runs the issue loop, waits included; an elected lane issues
        const uint32_t d_tmem = tmem_base + issuer * uint32_t(p.acc_cols);
        const uint32_t idesc = make_idesc_tf32(n_groups * 32, true, true, kPair ? 256u : 128u);
        // 8 pixels per MMA = two 512-byte groups of 4 rows (1 KB, 64 sixteen-byte units, per MMA); descriptors differ
        // only in the address field of their low word
        const uint64_t desc0 = make_smem_desc(smem_u32(smem), group_bytes, 512, kSwizzle128B_Atom32B);
        const uint32_t hi = uint32_t(desc0 >> 32), ring_lo0 = uint32_t(desc0);
        const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
        const uint32_t stage16 = stage_bytes >> 4, step16 = step_bytes >> 4, a16 = a_bytes >> 4;
        uint32_t full_a = full0 + 8u * issuer, empty_a = empty0 + 8u * issuer, slot_lo = ring_lo0 + issuer * stage16;
        const bool wide = p.pix == 64;
        // xhalo: N = 32*S per MMA, B's leading-dimension offset one 128-byte row (8 sixteen-byte units, bits 16-29 of
        // the low word) = one tap; a box row of bw pixels is bw/8 MMA steps per map group, the next box row starts
        // bw + S - 1 rows further in the haloed box
        const uint32_t idesc_x = make_idesc_tf32(p.S * 32, true, true, 128u);
        const uint32_t xn = p.S * 32, xg16 = uint32_t(p.x_group_bytes) >> 4;
        const uint32_t xlbo = (8u << 16) - (ring_lo0 & 0x3FFF0000u);      // replaces dy's offset field by 8
        const int xrows = p.pix >> p.bw_log2, xsteps = bw >> 3;
        const uint32_t xrow16 = uint32_t(bw + p.S - 1) * 8u;
        int stage = int(issuer);
        uint32_t phase = 0, accum = 0;
        bool ok = true;
        auto next_slot = [&]() {        // this thread's next slot: nis slots further round the ring
            stage += int(nis); full_a += 8u * nis; empty_a += 8u * nis; slot_lo += nis * stage16;
            if (stage >= p.stages) {
                stage -= p.stages; phase ^= 1u;
                full_a = full0 + 8u * stage; empty_a = empty0 + 8u * stage; slot_lo = ring_lo0 + uint32_t(stage) * stage16;
            }
        };
        // haloed x: one k-step per slot (KS = 1); the whole k-step is straight-line for the common box shapes
        auto xhalo_loop = [&](auto rows_c, auto steps_c, auto cg_c) {
            constexpr int kRows = decltype(rows_c)::value, kSteps = decltype(steps_c)::value, kCg = decltype(cg_c)::value;
            const int rows = kRows ? kRows : xrows, steps = kSteps ? kSteps : xsteps, cgs = kCg ? kCg : p.cg;
            for (int kit = int(issuer); kit < kiters; kit += int(nis)) {
                if (!bounded_wait_addr_warp(full_a, phase, &abort_flag, p.status, WAIT_MMA_FULL)) { ok = false; break; }
                tc_fence_after();
                uint32_t ar = slot_lo, br = slot_lo + a16 + xlbo;
                if constexpr (kRows != 0) {
#pragma unroll
                    for (int r = 0; r < kRows; ++r, ar += 64u * kSteps, br += xrow16)
                        xhalo_row<kSteps, kCg>(d_tmem, xn, ar, br, hi, idesc_x, r == 0 ? accum : 1u, xg16);
                } else {
                    for (int r = 0; r < rows; ++r, ar += 64u * steps, br += xrow16)
                        for (int m = 0; m < steps; ++m)
                            for (int g = 0; g < cgs; ++g)
                                umma_tf32(d_tmem + g * xn, (uint64_t(hi) << 32) | (ar + 64u * m),
                                          (uint64_t(hi) << 32) | (br + 64u * m + g * xg16), idesc_x, (accum | r | m) ? 1u : 0u);
                }
                accum = 1;
                umma_commit_addr<kPair>(empty_a);
                next_slot();
            }
        };
        using std::integral_constant;
        if (p.xhalo) {
            const int key = xrows * 100 + xsteps * 10 + p.cg;
            if (key == 422) xhalo_loop(integral_constant<int, 4>{}, integral_constant<int, 2>{}, integral_constant<int, 2>{});
            else if (key == 812) xhalo_loop(integral_constant<int, 8>{}, integral_constant<int, 1>{}, integral_constant<int, 2>{});
            else if (key == 242) xhalo_loop(integral_constant<int, 2>{}, integral_constant<int, 4>{}, integral_constant<int, 2>{});
            else if (key == 421) xhalo_loop(integral_constant<int, 4>{}, integral_constant<int, 2>{}, integral_constant<int, 1>{});
            else if (key == 222) xhalo_loop(integral_constant<int, 2>{}, integral_constant<int, 2>{}, integral_constant<int, 2>{});
            else xhalo_loop(integral_constant<int, 0>{}, integral_constant<int, 0>{}, integral_constant<int, 0>{});
        } else
        for (int kit = int(issuer) * p.KS; kit < kiters; kit += int(nis) * p.KS) {
            if (!bounded_wait_addr_warp(full_a, phase, &abort_flag, p.status, WAIT_MMA_FULL)) { ok = false; break; }
            tc_fence_after();
            const int nst = kiters - kit < p.KS ? kiters - kit : p.KS;
            uint32_t a_lo = slot_lo;
            for (int j = 0; j < nst; ++j, a_lo += step16) {
                umma_kstep_tf32<kPair, 64, 64>(d_tmem, a_lo, a_lo + a16, hi, hi, idesc, accum);
                accum = 1;
                if (wide) umma_kstep_tf32<kPair, 64, 64>(d_tmem, a_lo + 256, a_lo + a16 + 256, hi, hi, idesc, 1);
            }
            umma_commit_addr<kPair>(empty_a);
            next_slot();
        }
        if (ok) umma_commit_addr<kPair>(smem_u32(&tmem_full_bar));
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int k = kt * 128 + quarter * 32 + lane;
        const bool valid = k < p.K;
        const bool vec_ok = (p.C & 3) == 0;
        float4 db_acc[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
        const int bgroup = (kWide && warp > kSecondIssuerWarp) ? 1 : 0;       // builder group (the second has no epilogue)
        const int bwarp = bgroup ? warp - (kSecondIssuerWarp + 1) : warp - 2;  // 0 .. 7 inside the group
        constexpr int kGroups = kWide ? 2 : 1;
        const int t = bwarp * 32 + lane;                     // 0 .. 255 among the group's warps
        int maps_here = p.K - kt * 128;                      // output maps of this k tile
        if (maps_here > 128) maps_here = 128;
        const int units = maps_here >> 2;                    // 4-map units of the tile (K % 4 == 0)
        if (p.dy_pool) {
            // ---------------------------------------------------- builds the dy tiles (pooled-dy launches)
            const int hw = bw >> 1, hh = bh >> 1;             // the box in pooled pixels (bw, bh are even)
            const int ppix = p.pix >> 2;
            const int items = ppix * units;                   // (pooled pixel, 4-map unit) items per k-step: <= 512
            const int P2 = p.P >> 1, Q2 = p.Q >> 1;
            const uint32_t ring0 = smem_u32(smem);
            int stage = bgroup, sub = 0;
            uint32_t phase = 0, dstA = ring0;
            // the group's k-steps: slots bgroup, bgroup + kGroups, ... of KS boxes each; (qi, pi, ni) walks two k-steps
            // ahead of the k-step being written (the fetch cursor)
            int fb = box_begin + bgroup * p.KS, fsub = 0;
            int qi = fb % p.boxes_q;
            int pi = (fb / p.boxes_q) % p.boxes_p;
            int ni = fb / (p.boxes_q * p.boxes_p);
            bool ok = true;
            // this thread's (at most two) items: pooled pixel j of the box and 4-map unit u, the same in every k-step
            int item_w[2], item_h[2], item_n[2];
            uint32_t rowoff[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int item = t + 256 * i;
                rowoff[i] = 0xFFFFFFFFu; item_w[i] = item_h[i] = item_n[i] = 0;
                if (item < items) {
                    const int j = item / units, u = item - j * units;
                    item_w[i] = j % hw; item_h[i] = (j / hw) % hh; item_n[i] = j / (hw * hh);
                    // first of the window's four rows in the tile, and the unit's place in it
                    rowoff[i] = uint32_t(((item_n[i] * bh + 2 * item_h[i]) * bw + 2 * item_w[i]) << 7) | uint32_t(u);
                }
            }
            // byte offsets, inside a k-step's dy tile, of the item's 16 bytes at the window's four positions
            uint32_t off[2][4];
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (uint32_t e = 0; e < 4; ++e) {
                    const uint32_t u = rowoff[i] & 127u, row = (rowoff[i] >> 7) + (e >> 1) * uint32_t(bw) + (e & 1u);
                    off[i][e] = (u >> 3) * group_bytes + row * 128u + (((u & 7u) ^ ((row & 3u) << 1)) << 4);
                }
            // the loads of k-step b + 2 are issued before k-step b is written: their latency (DRAM: the pooled gradient
            // was written by the previous kernel and is larger than L2) overlaps two whole k-steps
            auto fetch = [&](int fqi, int fpi, int fni, float4 (&fv)[2], uint32_t (&fc)[2]) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    fv[i] = make_float4(0.f, 0.f, 0.f, 0.f); fc[i] = 0u;
                    if (rowoff[i] == 0xFFFFFFFFu) continue;
                    const int qq = fqi * hw + item_w[i], pp = fpi * hh + item_h[i], n = fni * bn + item_n[i];
                    if (qq < Q2 && pp < P2 && n < p.N) {
                        const size_t idx = ((static_cast<size_t>(n) * P2 + pp) * Q2 + qq) * p.K + kt * 128 + (rowoff[i] & 127u) * 4;
                        fv[i] = __ldg(reinterpret_cast<const float4*>(p.dy_pool + idx));
                        fc[i] = __ldg(reinterpret_cast<const unsigned int*>(p.codes + idx));
                    }
                }
            };
            float4 v[2], vn[2], vnn[2];
            uint32_t c[2], cn[2], cnn[2];
            auto next_box = [&]() {             // the fetch cursor's next k-step of this group
                int step = 1;
                if (++fsub == p.KS) { fsub = 0; step += (kGroups - 1) * p.KS; }
                fb += step;
                for (int i = 0; i < step; ++i)
                    if (++qi == p.boxes_q) {
                        qi = 0;
                        if (++pi == p.boxes_p) { pi = 0; ++ni; }
                    }
            };
            if (fb < box_end) { fetch(qi, pi, ni, vn, cn); next_box(); }
            if (fb < box_end) { fetch(qi, pi, ni, vnn, cnn); next_box(); }
            for (int b = box_begin + bgroup * p.KS; b < box_end && ok;) {
#pragma unroll
                for (int i = 0; i < 2; ++i) { v[i] = vn[i]; c[i] = cn[i]; vn[i] = vnn[i]; cn[i] = cnn[i]; }
                if (fb < box_end) { fetch(qi, pi, ni, vnn, cnn); next_box(); }
                if (sub == 0) {
                    if (!bounded_wait_warp(&empty_bar[stage], phase ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) { ok = false; break; }
                    dstA = ring0 + stage * stage_bytes;
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    if (rowoff[i] == 0xFFFFFFFFu) continue;
                    const float vv[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                    float live[4];
                    uint32_t pos[4];
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        const uint32_t code = (c[i] >> (8 * m)) & 7u;
                        pos[m] = code & 3u;
                        live[m] = (p.relu_mask && code >= 4u) ? 0.f : vv[m];
                    }
                    db_acc[i].x += live[0]; db_acc[i].y += live[1]; db_acc[i].z += live[2]; db_acc[i].w += live[3];
#pragma unroll
                    for (int m = 0; m < 4; ++m) live[m] = to_tf32(live[m]);
#pragma unroll
                    for (uint32_t e = 0; e < 4; ++e)
                        st_shared_v4(dstA + off[i][e], pos[0] == e ? live[0] : 0.f, pos[1] == e ? live[1] : 0.f,
                                     pos[2] == e ? live[2] : 0.f, pos[3] == e ? live[3] : 0.f);
                }
                dstA += step_bytes;
                if (++sub == p.KS || b == box_end - 1) {
                    sub = 0;
                    fence_proxy_async_shared();          // the tensor core reads the tile through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&full_bar[stage]);
                    stage += kGroups;
                    if (stage >= p.stages) { stage -= p.stages; phase ^= 1u; }
                    b += 1 + (kGroups - 1) * p.KS;       // over the other group's slot
                } else {
                    ++b;
                }
            }
        }
        if (bounded_wait_warp(&tmem_full_bar, 0, &abort_flag, p.status, WAIT_EPI_TMEM_FULL)) {
            tc_fence_after();
            if (p.dy_pool && p.db_rows && rb == 0) {        // (every run block would report the same sums)
                // Bias gradient: every warp adds up, per 4-map unit and in a fixed order, what its own lanes
                // scattered, and writes one row [K] per (split, warp); the caller adds the rows.  (Warp-local on
                // purpose: no barrier between warps that a timed-out warp could leave the others waiting at.  The
                // pipeline's shared memory is idle by now; the 1 KB slots lie behind the epilogue's staging tiles.)
                float4* scratch = reinterpret_cast<float4*>(smem + 32768) + (bgroup * 8 + bwarp) * 64;
                scratch[lane] = db_acc[0];
                scratch[32 + lane] = db_acc[1];
                __syncwarp();
                if (lane < units) {
                    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int e = 0; e < 64; ++e) {
                        const int item = (e < 32 ? 0 : 256 - 32) + bwarp * 32 + e;      // lane e (e - 32) of this warp, slot 0 (1)
                        if (item % units == lane) {
                            const float4 a = scratch[e];
                            sum.x += a.x; sum.y += a.y; sum.z += a.z; sum.w += a.w;
                        }
                    }
                    float* row = p.db_rows + (static_cast<size_t>(split) * kPooledDbRows + bgroup * 8 + bwarp) * p.K + kt * 128 + lane * 4;
                    *reinterpret_cast<float4*>(row) = sum;
                    if (!kWide) *reinterpret_cast<float4*>(row + 8 * static_cast<size_t>(p.K)) = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                __syncwarp();
            }
            if (bgroup == 0) {
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const size_t krow = static_cast<size_t>(valid ? k : 0) * p.R * p.S;
            // Each lane owns one output-map row of the accumulator, but 32 columns of a row are 128 contiguous
            // bytes of dw: a chunk is transposed through a 4 KB staging tile per warp (the pipeline's shared
            // memory, idle by now: every copy has landed and every MMA has read it) and written 4 rows x 128
            // bytes per instruction.
            const uint32_t stg = smem_u32(smem) + (warp - 2) * 4096;
            const int cg = (lane & 7) * 4;
            for (int ch = (warp - 2) >> 2; ch < n_groups; ch += 2) {     // the quarter's two warps take alternate chunks
                int tap, c0;
                if (p.xhalo) {                          // columns: [map group][tap of kernel row rb]
                    tap = rb * p.S + ch % p.S;
                    c0 = (ch / p.S) * 32;
                } else {
                    const int run = run0 + ch / p.L;
                    if (run >= p.total_runs) break;     // (pair mode) columns of runs past the last tap
                    tap = run / p.runs_per_tap;
                    c0 = ((run - tap * p.runs_per_tap) * p.L + ch % p.L) * 32;
                }
                // (in-place update: the old weights of the chunk are fetched before the accumulator is read and staged, so
                // that their latency does not fall between the stores)
                constexpr bool sgd = kSgd;
                float4 wv[8];
                if (sgd && vec_ok && c0 + cg < p.C) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int kk = kt * 128 + quarter * 32 + (lane >> 3) + 4 * i;
                        wv[i] = kk < p.K ? *reinterpret_cast<const float4*>(p.out + (static_cast<size_t>(kk) * p.R * p.S + tap) * p.C + c0 + cg)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                uint32_t v[32];
                if (kiters > 0) {
                    tmem_ld_32x32(t_row + ch * 32, v);
                    tmem_ld_wait();
                    if (p.duo && kiters > p.KS) {      // the second issuer had at least one slot
                        uint32_t u[32];
                        tmem_ld_32x32(t_row + p.acc_cols + ch * 32, u);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(u[j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (vec_ok) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        st_shared_v4(stg + lane * 128 + ((j ^ (lane & 7)) * 16), __uint_as_float(v[4 * j]),
                                     __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    __syncwarp();
                    if (c0 + cg < p.C) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = (lane >> 3) + 4 * i;
                            const int kk = kt * 128 + quarter * 32 + rr;
                            const float4 o = ld_shared_v4(stg + rr * 128 + (((lane & 7) ^ (rr & 7)) * 16));
                            if (kk < p.K) {
                                float* dst = p.out + static_cast<size_t>(split) * p.split_stride +
                                             (static_cast<size_t>(kk) * p.R * p.S + tap) * p.C + c0 + cg;
                                if (p.use_atomics) {
                                    atomicAdd(dst, o.x); atomicAdd(dst + 1, o.y); atomicAdd(dst + 2, o.z); atomicAdd(dst + 3, o.w);
                                } else if (sgd) {
                                    *reinterpret_cast<float4*>(dst) = make_float4(fmaf(-p.lr, o.x, wv[i].x), fmaf(-p.lr, o.y, wv[i].y),
                                                                                  fmaf(-p.lr, o.z, wv[i].z), fmaf(-p.lr, o.w, wv[i].w));
                                } else {
                                    *reinterpret_cast<float4*>(dst) = o;
                                }
                            }
                        }
                    }
                    __syncwarp();
                } else if (valid && c0 < p.C) {
                    float* dst = p.out + static_cast<size_t>(split) * p.split_stride + (krow + tap) * p.C + c0;
                    if (p.use_atomics) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < p.C) atomicAdd(dst + j, __uint_as_float(v[j]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < p.C) dst[j] = sgd ? fmaf(-p.lr, __uint_as_float(v[j]), dst[j]) : __uint_as_float(v[j]);
                    }
                }
            }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync_all();     // neither CTA leaves while the pair's MMAs may read its tiles
    if (warp == 1) {
        tc_fence_after();
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, p.tmem_cols);
        else tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// min_l: smallest log2 of the box width and height (1 for pooled dy: the box must hold whole 2x2 windows)
// min_lw: smallest log2 of the box width alone (3 for haloed x: a box row must hold whole 8-pixel MMA steps)
// stride_w / stride_h: the x box spans bw * stride_w x bh * stride_h input pixels, at most 256 each
void choose_pixel_box(int pix, int P, int Q, int N, int* bw_log2, int* bh_log2, int min_l = 0, int min_lw = 0,
                      int stride_w = 1, int stride_h = 1) {
    const int lp = pix == 64 ? 6 : 5;
    double best = 1e300;
    if (min_lw < min_l) min_lw = min_l;
    int best_w = min_lw, best_h = min_l;
    for (int lw = lp - min_l; lw >= min_lw; --lw)
        for (int lh = lp - lw; lh >= min_l; --lh) {
            const long bw = 1L << lw, bh = 1L << lh, bn = pix / (bw * bh);
            if (bw * stride_w > 256 || bh * stride_h > 256) continue;
            const double covered = double((Q + bw - 1) / bw * bw) * double((P + bh - 1) / bh * bh) *
                                   double((N + bn - 1) / bn * bn);
            if (covered < best) { best = covered; best_w = lw; best_h = lh; }
        }
    *bw_log2 = best_w;
    *bh_log2 = best_h;
}

// How a layer is cut into work items and k-steps.
struct WgradPlan {
    int grouped, L, runs_per_tap, total_runs, rpi, run_blocks;
    int pair;               // CTA pairs over k tiles 2i, 2i + 1
    int pix;                // pixels per k-step
    int KS, stages, step_bytes;
    int bw_log2, bh_log2;
    long boxes;
    int xhalo, x_group_bytes;     // haloed x boxes (see the header): item = (k tile, kernel row, split)
    int dy_groups;                // 32-map groups of the dy tile
};

WgradPlan plan_wgrad(int N, int P, int Q, int C, int K, int R, int S, int tap_groups, int pooled_dy = 0,
                     int stride_w = 1, int stride_h = 1, int dil_w = 1) {
    const bool strided = stride_w != 1 || stride_h != 1 || dil_w != 1;
    WgradPlan r{};
    const int cgroups = (C + 31) / 32;
    const int k_tiles = (K + 127) / 128;
    r.grouped = (!tap_groups && C % 32 == 0 && K % 32 == 0) ? 1 : 0;
    r.pair = tune(TUNE_PAIR_WGRAD, 1) && r.grouped && k_tiles % 2 == 0 && !pooled_dy;
    r.L = 1;
    if (r.grouped)
        for (int l = r.pair ? 4 : 8; l >= 1; --l)        // pair: each CTA loads whole runs, half of the item's
            if (cgroups % l == 0) { r.L = l; break; }
    r.runs_per_tap = cgroups / r.L;
    r.total_runs = R * S * r.runs_per_tap;
    const int rpi_max = 8 / r.L;
    if (tap_groups) {
        r.rpi = r.total_runs;                        // all tap rows of a k tile in one item
    } else {
        const int blocks = (r.total_runs + rpi_max - 1) / rpi_max;
        r.rpi = (r.total_runs + blocks - 1) / blocks;   // balanced: 18 runs -> 3 x 6 rather than 8 + 8 + 2
        if (r.pair && (r.rpi & 1)) ++r.rpi;             // (8 / L is even for L = 1..4, so this stays <= rpi_max)
    }
    r.run_blocks = (r.total_runs + r.rpi - 1) / r.rpi;
    // Haloed x boxes for single-CTA items of layers with few input maps (all taps of a kernel row fit one
    // accumulator): the pixel box must hold whole 8-pixel runs in w.
    if (r.grouped && !r.pair && !pooled_dy && !strided && S >= 2 && cgroups * S * 32 <= 256 && Q >= 8 && tune(TUNE_XHALO_WGRAD, 1)) {
        for (int pix = tune(TUNE_PIX_WGRAD, 64) == 64 ? 64 : 32; pix >= 32 && !r.xhalo; pix >>= 1) {
            int lw, lh;
            choose_pixel_box(pix, P, Q, N, &lw, &lh, 0, 3);
            const long bw = 1L << lw, bh = 1L << lh, bn = pix / (bw * bh);
            const int xg = int((bw + S - 1) * bh * bn * 128);
            const int step = (4 * pix * 128 + cgroups * xg + 1023) / 1024 * 1024;
            if (kSmemBudget / step < 3) continue;
            r.xhalo = 1; r.x_group_bytes = xg; r.pix = pix; r.step_bytes = step; r.dy_groups = 4;
            r.bw_log2 = lw; r.bh_log2 = lh;
            r.run_blocks = R;
            r.KS = 1;
            r.stages = kSmemBudget / step;
            if (r.stages > kMaxStages) r.stages = kMaxStages;
            r.boxes = ((Q + bw - 1) / bw) * ((P + bh - 1) / bh) * ((N + bn - 1) / bn);
        }
        if (r.xhalo) return r;
    }
    // 64-pixel k-steps halve the copies and commits per MMA; taken when three pipeline slots still fit
    const int x_groups = (r.pair ? r.rpi / 2 : r.rpi) * r.L;
    r.dy_groups = 4;
    if (pooled_dy && K < 128 && (K + 31) / 32 + x_groups >= 4) r.dy_groups = (K + 31) / 32;
    const int cta_groups = r.dy_groups + x_groups;      // 32-map groups a CTA loads per k-step
    r.pix = tune(TUNE_PIX_WGRAD, 64);
    if (r.pix != 64 || kSmemBudget / (cta_groups * 64 * 128) < 3) r.pix = 32;
    r.step_bytes = cta_groups * r.pix * 128;
    // A k-step of a narrow column block is a few short MMAs; such blocks get several k-steps per slot (one
    // barrier round trip and commit per slot) while at least 3 slots fit.
    const int max_groups = r.rpi * r.L;
    const int mma_clk = (r.pix / 8) * (max_groups * 16 > 52 ? max_groups * 16 : 52);
    r.KS = (600 + mma_clk - 1) / mma_clk;
    r.KS = tune(TUNE_KS_WGRAD, r.KS);
    while (r.KS > 1 && kSmemBudget / (r.KS * r.step_bytes) < 3) --r.KS;
    if (r.KS < 1) r.KS = 1;
    r.stages = kSmemBudget / (r.KS * r.step_bytes);
    if (r.stages > kMaxStages) r.stages = kMaxStages;
    choose_pixel_box(r.pix, P, Q, N, &r.bw_log2, &r.bh_log2, pooled_dy ? 1 : 0, 0, stride_w, stride_h);
    const long bw = 1L << r.bw_log2, bh = 1L << r.bh_log2, bn = r.pix / (bw * bh);
    r.boxes = ((Q + bw - 1) / bw) * ((P + bh - 1) / bh) * ((N + bn - 1) / bn);
    return r;
}

int sm_count() { return device_sm_count(); }

}  // namespace

bool tc_wgrad_eligible(const TcWgradArgs& a) {
    if (a.C % 4 != 0 || a.K % 4 != 0) return false;
    if (a.tap_groups && (a.S != 1 || a.C > 32 || a.R * 32 > 256)) return false;
    if (a.stride_h < 1 || a.stride_w < 1 || a.stride_h > 8 || a.stride_w > 8 || a.dil_w < 1) return false;
    if ((a.stride_h != 1 || a.stride_w != 1 || a.dil_w != 1) && (a.tap_groups || a.dy_pool)) return false;
    if ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.dy)) & 15) return false;
    return true;
}

bool tc_wgrad_can_take_pooled_dy(int N, int P, int Q, int C, int K, int R, int S, int tap_groups) {
    if (P % 2 != 0 || Q % 2 != 0 || K % 4 != 0 || N <= 0) return false;
    const WgradPlan rp = plan_wgrad(N, P, Q, C, K, R, S, tap_groups, 1);
    // the bias-gradient scratch (16 KB behind the epilogue's 32 KB of staging tiles) lies in the pipeline's memory
    return !rp.pair && (rp.stages & ~1) * rp.KS * rp.step_bytes >= 49152;
}

int tc_wgrad_splits(int N, int P, int Q, int C, int K, int R, int S, int tap_groups, int pooled_dy, int strided) {
    // (the number of work items and pixel boxes does not depend on the stride values, only on whether the haloed-x
    // form, which needs unit strides, is open)
    const WgradPlan rp = plan_wgrad(N, P, Q, C, K, R, S, tap_groups, pooled_dy, strided ? 2 : 1, strided ? 2 : 1);
    const long items = long((K + 127) / 128) * rp.run_blocks;
    long splits = sm_count() / items;
    if (splits < 1) splits = 1;
    if (splits > 64 && !tap_groups) splits = 64;
    if (splits > rp.boxes) splits = rp.boxes;
    // drop splits that would be empty
    const long per = (rp.boxes + splits - 1) / splits;
    splits = (rp.boxes + per - 1) / per;
    return int(splits);
}

namespace {
// What a launch needs that follows from its arguments alone; kept per distinct argument set like the forward-type
// kernel's plans (same key discipline: every field, the device, the generation of the tuning knobs).
struct WgradLaunchPlan {
    WgradParams p;
    CUtensorMap tmDy, tmX;
    bool pair = false, wide = false, zero_first = false;
    long items = 0;
    size_t smem = 0, dw_elems = 0;
    double flops = 0.0;
};
int build_wgrad_plan(const TcWgradArgs& a, WgradLaunchPlan* plan);
int run_wgrad_plan(const WgradLaunchPlan& plan, const TcWgradArgs& a, cudaStream_t st);
std::string wgrad_plan_key(const TcWgradArgs& a, int device) {
    std::string k;
    k.reserve(256);
    auto put = [&k](const void* v, size_t n) { k.append(static_cast<const char*>(v), n); };
    const void* ptrs[] = {a.x, a.dy, a.dw, a.partial, a.dy_pool, a.codes, a.db_rows, a.w_update};
    put(ptrs, sizeof(ptrs));
    const int ints[] = {a.N, a.H, a.W, a.C, a.K, a.R, a.S, a.pad_h, a.pad_w, a.P, a.Q, a.splits, a.x_inner, a.tap_groups, a.skip_reduce,
                        a.relu_mask, a.stride_h, a.stride_w, a.dil_w, device};
    put(ints, sizeof(ints));
    const long longs[] = {a.x_stride_w, a.x_stride_h, a.x_stride_n};
    put(longs, sizeof(longs));
    put(&a.lr, sizeof(a.lr));
    const unsigned gen = tune_generation();
    put(&gen, sizeof(gen));
    return k;
}
std::mutex g_wplan_mu;
std::unordered_map<std::string, WgradLaunchPlan> g_wplans;
}  // namespace

int launch_tc_wgrad(const TcWgradArgs& a, cudaStream_t st) {
    WgradLaunchPlan plan;
    if (!tune(TUNE_PLAN_CACHE, 1)) {
        const int rc = build_wgrad_plan(a, &plan);
        return rc != PCL_OK ? rc : run_wgrad_plan(plan, a, st);
    }
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return PCL_ERR_CUDA;
    const std::string key = wgrad_plan_key(a, device);
    bool hit = false;
    {
        std::lock_guard<std::mutex> lock(g_wplan_mu);
        auto it = g_wplans.find(key);
        if (it != g_wplans.end()) { plan = it->second; hit = true; }
    }
    if (!hit) {
        const int rc = build_wgrad_plan(a, &plan);
        if (rc != PCL_OK) return rc;
        std::lock_guard<std::mutex> lock(g_wplan_mu);
        if (g_wplans.size() >= 512) g_wplans.clear();
        g_wplans.emplace(key, plan);
    }
    plan_cache_count(hit);
    return run_wgrad_plan(plan, a, st);
}

namespace {
int build_wgrad_plan(const TcWgradArgs& a, WgradLaunchPlan* plan) {
    if (!tc_wgrad_eligible(a)) return PCL_ERR_UNSUPPORTED_SHAPE;
    static PerDeviceOnce attr_once;       // (the attribute applies to the current device only)
    const int setup_rc = attr_once.run([]() -> int {
        if (cudaFuncSetAttribute(tc_wgrad_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(tc_wgrad_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(tc_wgrad_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(tc_wgrad_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(tc_wgrad_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBudget + 1024) != cudaSuccess)
            return PCL_ERR_CUDA;
        return PCL_OK;
    });
    if (setup_rc != PCL_OK) return setup_rc;
    WgradParams p{};
    const int pooled = a.dy_pool ? 1 : 0;
    if (pooled && (!a.codes || !tc_wgrad_can_take_pooled_dy(a.N, a.P, a.Q, a.C, a.K, a.R, a.S, a.tap_groups)))
        return PCL_ERR_UNSUPPORTED_SHAPE;
    const WgradPlan rp = plan_wgrad(a.N, a.P, a.Q, a.C, a.K, a.R, a.S, a.tap_groups, pooled, a.stride_w, a.stride_h, a.dil_w);
    p.dy_pool = a.dy_pool; p.codes = a.codes; p.relu_mask = a.relu_mask; p.db_rows = pooled ? a.db_rows : nullptr;
    p.N = a.N; p.P = a.P; p.Q = a.Q;
    p.pix = rp.pix; p.bw_log2 = rp.bw_log2; p.bh_log2 = rp.bh_log2;
    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2, bn = p.pix / (bw * bh);
    p.boxes_q = (a.Q + bw - 1) / bw;
    p.boxes_p = (a.P + bh - 1) / bh;
    p.boxes_n = (a.N + bn - 1) / bn;
    const long boxes = rp.boxes;
    if (boxes > 0x7fffffffL) return PCL_ERR_UNSUPPORTED_SHAPE;
    p.xhalo = rp.xhalo; p.cg = (a.C + 31) / 32; p.x_group_bytes = rp.x_group_bytes; p.x_step_bytes = rp.step_bytes;
    p.grouped = rp.grouped; p.grouped_dy = (a.K % 32 == 0) ? 1 : 0; p.x_taprows = a.tap_groups ? 1 : 0; p.L = rp.L; p.runs_per_tap = rp.runs_per_tap; p.total_runs = rp.total_runs;
    p.rpi = rp.rpi; p.run_blocks = rp.run_blocks;
    p.k_tiles = (a.K + 127) / 128;
    p.R = a.R; p.S = a.S; p.pad_h = a.pad_h; p.pad_w = a.pad_w;
    p.stride_h = a.stride_h; p.stride_w = a.stride_w; p.dil_w = a.dil_w;
    p.K = a.K; p.C = a.C;
    p.splits = a.splits;
    if (p.splits < 1) return PCL_ERR_BAD_ARG;
    p.boxes_per_split = int((boxes + p.splits - 1) / p.splits);
    const int max_groups = p.xhalo ? p.cg * a.S : p.rpi * p.L;
    p.KS = rp.KS; p.stages = rp.stages;
    const int stage_bytes = p.KS * rp.step_bytes;
    p.dy_groups = rp.dy_groups;
    p.acc_cols = max_groups * 32;
    p.duo = (!rp.pair && p.stages >= 4 && 2 * p.acc_cols <= 512 && tune(TUNE_ISSUERS, 2) >= 2) ? 1 : 0;
    if (p.duo) p.stages &= ~1;      // an even ring: every slot stays with one issuing thread
    p.tmem_cols = 32;
    while (p.tmem_cols < (p.duo ? 2 : 1) * p.acc_cols) p.tmem_cols *= 2;
    p.status = device_status_ptr();
    if (!p.status) return PCL_ERR_CUDA;
    p.inject_short_copy = (tune(TUNE_FAULT_INJECT, 0) == 2 && !rp.pair && !pooled) ? 1 : 0;      // test mode
    const size_t dw_elems = size_t(a.K) * a.R * a.S * a.C;
    bool zero_first = false;
    if (a.w_update && p.splits != 1) return PCL_ERR_BAD_ARG;      // (a split reduction updates in its second pass)
    if (p.splits == 1) {
        p.out = a.w_update ? a.w_update : a.dw; p.split_stride = 0; p.use_atomics = 0;
        p.sgd = a.w_update ? 1 : 0; p.lr = a.lr;
    } else if (a.partial) {
        p.out = a.partial; p.split_stride = dw_elems; p.use_atomics = 0;
    } else {
        p.out = a.dw; p.split_stride = 0; p.use_atomics = 1;
        zero_first = true;
    }

    // When both map counts are multiples of 32, each tensor is viewed as 5-D {32 maps, w, h, n, group} (the
    // group dimension has a 128-byte stride) so that one TMA instruction brings a whole run of groups, laid
    // out [group][pixel][32 maps] in shared memory exactly as per-group boxes would be.
    CUtensorMap tmDy, tmX;
    if (!pooled) {
        const uint64_t sw = uint64_t(a.K), sh = uint64_t(a.Q) * a.K, sn = uint64_t(a.P) * a.Q * a.K;
        if (p.grouped_dy) {
            const uint64_t dims[5] = {32, uint64_t(a.Q), uint64_t(a.P), uint64_t(a.N), uint64_t(a.K / 32)};
            const uint64_t strides[4] = {sw * 4, sh * 4, sn * 4, 128};
            const uint32_t box[5] = {32, uint32_t(bw), uint32_t(bh), uint32_t(bn), 4};
            int rc = make_tmap(&tmDy, a.dy, 5, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        } else {
            const uint64_t dims[4] = {uint64_t(a.K), uint64_t(a.Q), uint64_t(a.P), uint64_t(a.N)};
            const uint64_t strides[3] = {sw * 4, sh * 4, sn * 4};
            const uint32_t box[4] = {32, uint32_t(bw), uint32_t(bh), uint32_t(bn)};
            int rc = make_tmap(&tmDy, a.dy, 4, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        }
    }
    {
        const uint64_t sw = a.x_stride_w ? uint64_t(a.x_stride_w) : uint64_t(a.C);
        const uint64_t sh = a.x_stride_h ? uint64_t(a.x_stride_h) : uint64_t(a.W) * a.C;
        const uint64_t sn = a.x_stride_n ? uint64_t(a.x_stride_n) : uint64_t(a.H) * a.W * a.C;
        if (p.xhalo) {
            // haloed box: S - 1 more columns than the dy box, all map groups with one instruction
            const uint64_t dims[5] = {32, uint64_t(a.W), uint64_t(a.H), uint64_t(a.N), uint64_t(a.C / 32)};
            const uint64_t strides[4] = {sw * 4, sh * 4, sn * 4, 128};
            const uint32_t box[5] = {32, uint32_t(bw + a.S - 1), uint32_t(bh), uint32_t(bn), uint32_t(p.cg)};
            int rc = make_tmap(&tmX, a.x, 5, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        } else if (p.x_taprows) {
            // few-channel path: the R tap rows of a pixel window are R boxes one image row apart; a 5th
            // dimension with the row stride fetches them with one instruction (H extent shrinks by R-1 so
            // that row + tap stays inside the staged image)
            const uint64_t dims[5] = {uint64_t(a.x_inner ? a.x_inner : a.C), uint64_t(a.W), uint64_t(a.H - a.R + 1),
                                      uint64_t(a.N), uint64_t(a.R)};
            const uint64_t strides[4] = {sw * 4, sh * 4, sn * 4, sh * 4};
            const uint32_t box[5] = {32, uint32_t(bw), uint32_t(bh), uint32_t(bn), uint32_t(a.R)};
            int rc = make_tmap(&tmX, a.x, 5, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        } else if (p.grouped) {
            const uint64_t dims[5] = {32, uint64_t(a.W), uint64_t(a.H), uint64_t(a.N), uint64_t(a.C / 32)};
            const uint64_t strides[4] = {sw * 4, sh * 4, sn * 4, 128};
            const uint32_t box[5] = {32, uint32_t(bw * a.stride_w), uint32_t(bh * a.stride_h), uint32_t(bn), uint32_t(p.L)};
            const uint32_t estr[5] = {1, uint32_t(a.stride_w), uint32_t(a.stride_h), 1, 1};
            int rc = make_tmap(&tmX, a.x, 5, dims, strides, box, true, false, estr);
            if (rc != PCL_OK) return rc;
        } else {
            const uint64_t dims[4] = {uint64_t(a.x_inner ? a.x_inner : a.C), uint64_t(a.W), uint64_t(a.H),
                                      uint64_t(a.N)};
            const uint64_t strides[3] = {sw * 4, sh * 4, sn * 4};
            const uint32_t box[4] = {32, uint32_t(bw * a.stride_w), uint32_t(bh * a.stride_h), uint32_t(bn)};
            const uint32_t estr[4] = {1, uint32_t(a.stride_w), uint32_t(a.stride_h), 1};
            int rc = make_tmap(&tmX, a.x, 4, dims, strides, box, true, false, estr);
            if (rc != PCL_OK) return rc;
        }
    }
    if (pooled) tmDy = tmX;      // (a valid map is passed in any case; the kernel does not use it)
    const long items = long(p.k_tiles) * p.run_blocks * p.splits;
    if (items > 0x7fffffffL) return PCL_ERR_UNSUPPORTED_SHAPE;
    const size_t smem = size_t(p.stages) * stage_bytes + 1024;
    plan->p = p; plan->tmDy = tmDy; plan->tmX = tmX;
    plan->pair = rp.pair != 0; plan->wide = pooled && p.duo; plan->zero_first = zero_first;
    plan->items = items; plan->smem = smem; plan->dw_elems = dw_elems;
    plan->flops = 2.0 * a.N * a.P * a.Q * double(a.K) * a.C * a.R * a.S;
    return PCL_OK;
}

int run_wgrad_plan(const WgradLaunchPlan& plan, const TcWgradArgs& a, cudaStream_t st) {
    const WgradParams& p = plan.p;
    const CUtensorMap& tmDy = plan.tmDy;
    const CUtensorMap& tmX = plan.tmX;
    const long items = plan.items;
    const size_t smem = plan.smem, dw_elems = plan.dw_elems;
    if (plan.zero_first) {
        const int rc = launch_zero(a.dw, dw_elems, st);
        if (rc != PCL_OK) return rc;
    }
    {
        LaunchScope scope(KID_TC_WGRAD, plan.flops, st);
        if (plan.pair) {
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cudaLaunchConfig_t lc{};
            lc.gridDim = dim3(unsigned(items)); lc.blockDim = dim3(kWgradThreads); lc.dynamicSmemBytes = smem; lc.stream = st;
            lc.attrs = attr; lc.numAttrs = 1;
            const cudaError_t le = p.sgd ? cudaLaunchKernelEx(&lc, tc_wgrad_kernel<true, false, true>, tmDy, tmX, p)
                                         : cudaLaunchKernelEx(&lc, tc_wgrad_kernel<true>, tmDy, tmX, p);
            if (le != cudaSuccess) return PCL_ERR_CUDA;
        } else if (plan.wide) {
            tc_wgrad_kernel<false, true><<<int(items), kWgradThreadsWide, smem, st>>>(tmDy, tmX, p);
        } else if (p.sgd) {
            tc_wgrad_kernel<false, false, true><<<int(items), kWgradThreads, smem, st>>>(tmDy, tmX, p);
        } else {
            tc_wgrad_kernel<false><<<int(items), kWgradThreads, smem, st>>>(tmDy, tmX, p);
        }
    }
    if (cudaGetLastError() != cudaSuccess) return PCL_ERR_CUDA;
    if (p.splits > 1 && a.partial && !a.skip_reduce) return launch_reduce_splits(a.partial, a.dw, dw_elems, p.splits, st);
    return PCL_OK;
}
}  // namespace

}  // namespace pcl
