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
#include <stdlib.h>

#include "pcl_internal.h"
#include "pcl_ptx.cuh"

namespace pcl {

namespace {

constexpr int kPix = 32;              // pixels (reduction indices) per pipeline slot
constexpr int kGroupBytes = kPix * 128;   // one {32 maps x 32 pixels} box
constexpr int kABytes = 4 * kGroupBytes;  // 128 output maps
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 224 * 1024;

struct WgradParams {
    int bw_log2, bh_log2;     // pixel box bw x bh x (32/(bw*bh))
    int boxes_q, boxes_p, boxes_n;
    int k_tiles;
    int L;                    // 32-map groups per run
    int runs_per_tap;         // ceil(C/32) / L
    int total_runs;           // R*S*runs_per_tap
    int rpi;                  // runs per work item (rpi*L <= 8)
    int run_blocks;           // ceil(total_runs / rpi)
    int R, S, pad_h, pad_w;
    int K, C;
    int splits, boxes_per_split;
    int stages, tmem_cols;
    int KS;                   // pixel boxes (k-steps of 32 pixels) per pipeline slot; > 1 for narrow column blocks
    int use_atomics;
    int grouped;              // x: 5-D tensor map (one TMA instruction per run) or 4-D per-group boxes (L == 1)
    int grouped_dy;           // dy: 5-D tensor map (all four 32-map groups in one instruction)
    int x_taprows;            // x: 5-D map whose 5th dimension is the tap row (few-channel path): one instruction per k-step
    float* out;               // dw, or the partial-sum workspace [splits][K*R*S*C]
    size_t split_stride;      // K*R*S*C (0 when writing straight to dw)
    unsigned int* status;     // device status word
};

__global__ void __launch_bounds__(192, 1)
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

    // work item of this CTA
    int item = blockIdx.x;
    const int split = item % p.splits;   item /= p.splits;
    const int rb = item % p.run_blocks;
    const int kt = item / p.run_blocks;
    const int run0 = rb * p.rpi;
    const int nruns = (run0 + p.rpi <= p.total_runs) ? p.rpi : p.total_runs - run0;
    const int n_groups = nruns * p.L;                 // 32-column groups of this item's MMA
    const uint32_t step_bytes = kABytes + p.rpi * p.L * kGroupBytes;    // one k-step (same for every item)
    const uint32_t stage_bytes = p.KS * step_bytes;                     // a slot holds KS k-steps
    const uint32_t tx_bytes = kABytes + n_groups * kGroupBytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&tmem_full_bar, 1);
        abort_flag = 0;
        mbar_fence_init();
        prefetch_tmap(&tmDy);
        prefetch_tmap(&tmX);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_slot, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    const int total_boxes = p.boxes_q * p.boxes_p * p.boxes_n;
    const int box_begin = split * p.boxes_per_split;
    int box_end = box_begin + p.boxes_per_split;
    if (box_end > total_boxes) box_end = total_boxes;
    const int kiters = box_end > box_begin ? box_end - box_begin : 0;
    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2, bn = kPix >> (p.bw_log2 + p.bh_log2);

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            // Per-run TMA coordinates are fixed for the item: decode them once (the k loop must stay
            // free of integer divisions, this thread paces the whole pipeline).
            int run_dw[8], run_dh[8], run_c[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int run = run0 + (j < nruns ? j : 0);
                const int tap = run / p.runs_per_tap;
                const int cg0 = (run - tap * p.runs_per_tap) * p.L;
                const int r = tap / p.S, s = tap - r * p.S;
                run_dw[j] = s - p.pad_w;
                run_dh[j] = r - p.pad_h;
                run_c[j] = p.grouped ? cg0 : cg0 * 32;
            }
            int qi = box_begin % p.boxes_q;
            int pi = (box_begin / p.boxes_q) % p.boxes_p;
            int ni = box_begin / (p.boxes_q * p.boxes_p);
            const uint32_t run_bytes = p.L * kGroupBytes;
            int sub = 0;                                         // position of the k-step inside its slot
            for (int b = box_begin; b < box_end; ++b) {
                const int q0 = qi * bw, p0 = pi * bh, n0 = ni * bn;
                if (++qi == p.boxes_q) { qi = 0; if (++pi == p.boxes_p) { pi = 0; ++ni; } }
                if (sub == 0) {
                    if (!bounded_wait(&empty_bar[stage], phase ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) { ok = false; break; }
                    const int nst = box_end - b < p.KS ? box_end - b : p.KS;
                    mbar_expect_tx(&full_bar[stage], nst * tx_bytes);
                }
                uint8_t* dst = smem + stage * stage_bytes + sub * step_bytes;
                if (p.grouped_dy) {
                    tma_load_5d(dst, &tmDy, &full_bar[stage], 0, q0, p0, n0, kt * 4);
                } else {
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        tma_load_4d(dst + g * kGroupBytes, &tmDy, &full_bar[stage], kt * 128 + g * 32, q0, p0, n0);
                }
                if (p.x_taprows) {
                    tma_load_5d(dst + kABytes, &tmX, &full_bar[stage], 0, q0 + run_dw[0], p0 + run_dh[0], n0, 0);
                } else if (p.grouped) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < nruns)
                            tma_load_5d(dst + kABytes + j * run_bytes, &tmX, &full_bar[stage], 0, q0 + run_dw[j],
                                        p0 + run_dh[j], n0, run_c[j]);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j < nruns)
                            tma_load_4d(dst + kABytes + j * run_bytes, &tmX, &full_bar[stage], run_c[j],
                                        q0 + run_dw[j], p0 + run_dh[j], n0);
                }
                if (++sub == p.KS || b == box_end - 1) {
                    sub = 0;
                    ++issued;
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
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
    } else if (warp == 1) {
        if (lane == 0) {     // one thread runs the whole issue loop, waits included
        const uint32_t idesc = make_idesc_tf32(n_groups * 32, true, true);
        const uint64_t desc0 = make_smem_desc(0, kGroupBytes, 512, kSwizzle128B_Atom32B);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int kit = 0; kit < kiters; kit += p.KS) {
            if (!bounded_wait(&full_bar[stage], phase, &abort_flag, p.status, WAIT_MMA_FULL)) { ok = false; break; }
            tc_fence_after();
            const int nst = kiters - kit < p.KS ? kiters - kit : p.KS;
            {
              for (int j = 0; j < nst; ++j) {
                // 8 pixels per instruction = two 512-byte groups of 4 rows; descriptors differ only in the
                // address field, so add offsets to a constant part
                const uint64_t da = desc0 + ((smem_u32(smem + stage * stage_bytes + j * step_bytes) & 0x3FFFFu) >> 4);
                const uint64_t db = da + (kABytes >> 4);
#pragma unroll
                for (int kk = 0; kk < kPix / 8; ++kk)
                    umma_tf32(tmem_base, da + kk * (1024 >> 4), db + kk * (1024 >> 4), idesc, (kit | j | kk) != 0);
              }
                umma_commit(&empty_bar[stage]);
            }
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tmem_full_bar);
        }
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int k = kt * 128 + quarter * 32 + lane;
        const bool valid = k < p.K;
        const bool vec_ok = (p.C & 3) == 0;
        if (bounded_wait_warp(&tmem_full_bar, 0, &abort_flag, p.status, WAIT_EPI_TMEM_FULL)) {
            tc_fence_after();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const size_t krow = static_cast<size_t>(valid ? k : 0) * p.R * p.S;
            for (int ch = 0; ch < n_groups; ++ch) {
                const int run = run0 + ch / p.L;
                const int tap = run / p.runs_per_tap;
                const int c0 = ((run - tap * p.runs_per_tap) * p.L + ch % p.L) * 32;
                float* dst = p.out + static_cast<size_t>(split) * p.split_stride + (krow + tap) * p.C + c0;
                uint32_t v[32];
                if (kiters > 0) {
                    tmem_ld_32x32(t_row + ch * 32, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (valid && c0 < p.C) {
                    if (p.use_atomics) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < p.C) atomicAdd(dst + j, __uint_as_float(v[j]));
                    } else if (vec_ok) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c0 + j < p.C)
                                *reinterpret_cast<float4*>(dst + j) =
                                    make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < p.C) dst[j] = __uint_as_float(v[j]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

void choose_pixel_box(int P, int Q, int N, int* bw_log2, int* bh_log2) {
    double best = 1e300;
    int best_w = 0, best_h = 0;
    for (int lw = 5; lw >= 0; --lw)
        for (int lh = 5 - lw; lh >= 0; --lh) {
            const long bw = 1L << lw, bh = 1L << lh, bn = kPix / (bw * bh);
            const double covered = double((Q + bw - 1) / bw * bw) * double((P + bh - 1) / bh * bh) *
                                   double((N + bn - 1) / bn * bn);
            if (covered < best) { best = covered; best_w = lw; best_h = lh; }
        }
    *bw_log2 = best_w;
    *bh_log2 = best_h;
}

long total_pixel_boxes(int N, int P, int Q) {
    int lw, lh;
    choose_pixel_box(P, Q, N, &lw, &lh);
    const long bw = 1L << lw, bh = 1L << lh, bn = kPix / (bw * bh);
    return ((Q + bw - 1) / bw) * ((P + bh - 1) / bh) * ((N + bn - 1) / bn);
}

// How the columns of a layer are cut into runs and work items.
struct RunPlan {
    int grouped, L, runs_per_tap, total_runs, rpi, run_blocks;
};

RunPlan plan_runs(int C, int K, int R, int S, int tap_groups) {
    RunPlan r{};
    const int cgroups = (C + 31) / 32;
    r.grouped = (!tap_groups && C % 32 == 0 && K % 32 == 0) ? 1 : 0;
    r.L = 1;
    if (r.grouped)
        for (int l = 8; l >= 1; --l)
            if (cgroups % l == 0) { r.L = l; break; }
    r.runs_per_tap = cgroups / r.L;
    r.total_runs = R * S * r.runs_per_tap;
    const int rpi_max = 8 / r.L;
    if (tap_groups) {
        r.rpi = r.total_runs;                        // all tap rows of a k tile in one item
    } else {
        const int blocks = (r.total_runs + rpi_max - 1) / rpi_max;
        r.rpi = (r.total_runs + blocks - 1) / blocks;   // balanced: 18 runs -> 3 x 6 rather than 8 + 8 + 2
    }
    r.run_blocks = (r.total_runs + r.rpi - 1) / r.rpi;
    return r;
}

int g_sm_count = 0;
int sm_count() {
    if (g_sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_sm_count <= 0)
            g_sm_count = 148;   // sizing only; a launch would fail anyway without a device
    }
    return g_sm_count;
}
bool g_attr_set = false;

}  // namespace

bool tc_wgrad_eligible(const TcWgradArgs& a) {
    if (a.C % 4 != 0 || a.K % 4 != 0) return false;
    if (a.tap_groups && (a.S != 1 || a.C > 32 || a.R * 32 > 256)) return false;
    if ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.dy)) & 15) return false;
    return true;
}

int tc_wgrad_splits(int N, int P, int Q, int C, int K, int R, int S, int tap_groups) {
    const RunPlan rp = plan_runs(C, K, R, S, tap_groups);
    const long items = long((K + 127) / 128) * rp.run_blocks;
    const long boxes = total_pixel_boxes(N, P, Q);
    long splits = sm_count() / items;
    if (splits < 1) splits = 1;
    if (splits > 64 && !tap_groups) splits = 64;
    if (splits > boxes) splits = boxes;
    // drop splits that would be empty
    const long per = (boxes + splits - 1) / splits;
    splits = (boxes + per - 1) / per;
    return int(splits);
}

int launch_tc_wgrad(const TcWgradArgs& a, cudaStream_t st) {
    if (!tc_wgrad_eligible(a)) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!g_attr_set) {
        if (cudaFuncSetAttribute(tc_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024) !=
            cudaSuccess)
            return PCL_ERR_CUDA;
        g_attr_set = true;
    }
    WgradParams p{};
    choose_pixel_box(a.P, a.Q, a.N, &p.bw_log2, &p.bh_log2);
    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2, bn = kPix / (bw * bh);
    p.boxes_q = (a.Q + bw - 1) / bw;
    p.boxes_p = (a.P + bh - 1) / bh;
    p.boxes_n = (a.N + bn - 1) / bn;
    const long boxes = long(p.boxes_q) * p.boxes_p * p.boxes_n;
    if (boxes > 0x7fffffffL) return PCL_ERR_UNSUPPORTED_SHAPE;
    const RunPlan rp = plan_runs(a.C, a.K, a.R, a.S, a.tap_groups);
    p.grouped = rp.grouped; p.grouped_dy = (a.K % 32 == 0) ? 1 : 0; p.x_taprows = a.tap_groups ? 1 : 0; p.L = rp.L; p.runs_per_tap = rp.runs_per_tap; p.total_runs = rp.total_runs;
    p.rpi = rp.rpi; p.run_blocks = rp.run_blocks;
    p.k_tiles = (a.K + 127) / 128;
    p.R = a.R; p.S = a.S; p.pad_h = a.pad_h; p.pad_w = a.pad_w;
    p.K = a.K; p.C = a.C;
    p.splits = a.splits;
    p.boxes_per_split = int((boxes + p.splits - 1) / p.splits);
    const int max_groups = p.rpi * p.L;
    const int step_bytes = kABytes + max_groups * kGroupBytes;
    // A k-step of a narrow column block is 4 short MMAs; the issuing thread's per-slot round trip (~600
    // cycles) then dominates, so such blocks get several k-steps per slot while at least 3 slots fit.
    const int mma_clk = 4 * (max_groups * 16 > 52 ? max_groups * 16 : 52);
    p.KS = (600 + mma_clk - 1) / mma_clk;
    if (getenv("PCL_KS_WGRAD")) p.KS = atoi(getenv("PCL_KS_WGRAD"));
    while (p.KS > 1 && kSmemBudget / (p.KS * step_bytes) < 3) --p.KS;
    if (p.KS < 1) p.KS = 1;
    const int stage_bytes = p.KS * step_bytes;
    p.stages = kSmemBudget / stage_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    p.tmem_cols = 32;
    while (p.tmem_cols < max_groups * 32) p.tmem_cols *= 2;
    p.status = device_status_ptr();
    if (!p.status) return PCL_ERR_CUDA;
    const size_t dw_elems = size_t(a.K) * a.R * a.S * a.C;
    if (p.splits == 1) {
        p.out = a.dw; p.split_stride = 0; p.use_atomics = 0;
    } else if (a.partial) {
        p.out = a.partial; p.split_stride = dw_elems; p.use_atomics = 0;
    } else {
        p.out = a.dw; p.split_stride = 0; p.use_atomics = 1;
        int rc = launch_zero(a.dw, dw_elems, st);
        if (rc != PCL_OK) return rc;
    }

    // When both map counts are multiples of 32, each tensor is viewed as 5-D {32 maps, w, h, n, group} (the
    // group dimension has a 128-byte stride) so that one TMA instruction brings a whole run of groups, laid
    // out [group][pixel][32 maps] in shared memory exactly as per-group boxes would be.
    CUtensorMap tmDy, tmX;
    {
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
        if (p.x_taprows) {
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
            const uint32_t box[5] = {32, uint32_t(bw), uint32_t(bh), uint32_t(bn), uint32_t(p.L)};
            int rc = make_tmap(&tmX, a.x, 5, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        } else {
            const uint64_t dims[4] = {uint64_t(a.x_inner ? a.x_inner : a.C), uint64_t(a.W), uint64_t(a.H),
                                      uint64_t(a.N)};
            const uint64_t strides[3] = {sw * 4, sh * 4, sn * 4};
            const uint32_t box[4] = {32, uint32_t(bw), uint32_t(bh), uint32_t(bn)};
            int rc = make_tmap(&tmX, a.x, 4, dims, strides, box, true);
            if (rc != PCL_OK) return rc;
        }
    }
    const long items = long(p.k_tiles) * p.run_blocks * p.splits;
    if (items > 0x7fffffffL) return PCL_ERR_UNSUPPORTED_SHAPE;
    const size_t smem = size_t(p.stages) * stage_bytes + 1024;
    {
        LaunchScope scope(KID_TC_WGRAD, 2.0 * a.N * a.P * a.Q * double(a.K) * a.C * a.R * a.S, st);
        tc_wgrad_kernel<<<int(items), 192, smem, st>>>(tmDy, tmX, p);
    }
    if (cudaGetLastError() != cudaSuccess) return PCL_ERR_CUDA;
    if (p.splits > 1 && a.partial && !a.skip_reduce) return launch_reduce_splits(a.partial, a.dw, dw_elems, p.splits, st);
    return PCL_OK;
}

}  // namespace pcl
