// Forward-type implicit-GEMM convolution on the 5th-generation tensor cores.
//
//   out[n,p,q,k] = epi( sum_{r,s,c} in[n, p+r-pad_h, q+s-pad_w, c] * wt[k, r*S+s, c] )
//
// (Algorithm 1 with stride 1; the same kernel computes the backward-data pass of
// a stride-1 layer when it is handed dy as `in` and either the layer's own KRSC
// weights, read in place as an MN-major operand with the taps flipped by index,
// or a flipped, transposed copy; and the fully-connected GEMMs as the 1x1 /
// 1x1-map special case.)
//
// GEMM view: M = N*P*Q output pixels, N = Kout, reduction over (r, s, c).
// One CTA tile is 128 output pixels x BN output maps.  The 128 pixels are a
// box bw x bh x bn of the (q, p, n) index space, so that for a fixed tap (r, s)
// the A operand is one TMA box of the NHWC input shifted by the tap: the im2col
// matrix is never materialised and zero padding is TMA's out-of-bounds fill.
// B is a TMA box of BN weight rows.  Variants, chosen per launch on the host:
//   plain tiling    one box per tap; a slot holds two channel blocks fetched by one copy per operand
//   haloed tiling   one input patch per channel block, taps are row-shifted views of it (narrow layers)
//   CTA pairs       two CTAs of a cluster share a weight tile, the leader issues M = 256 MMAs (cta_group::2)
//
// Warp roles (352 threads, persistent over tiles):
//   warp 0        TMA producer, fills the ring of slots (the warp runs its loop converged, an elected lane issues)
//   warp 1        allocates TMEM; issues tcgen05.mma kind::tf32 (mma_issuer(); converged warp, elected lane)
//   warp 10       second issuing warp: alternate slots of single-CTA tiles with many slots, or alternate tiles of the
//                 few-channel first layer
//   warps 2-9     epilogue: TMEM -> registers -> bias / activation / mask [/ column sums / 2x2 max pool]
//                 -> global, through TMA stores or coalesced per-lane stores (two warps per TMEM lane quarter)
//   warps 11-18   eight more epilogue warps (608 threads) in the variant for tiles with a very short reduction
// Two TMEM accumulator sets let the epilogue of tile i overlap the main loop of tile i+1.
#include <stdio.h>
#include <stdlib.h>

#include <atomic>
#include <mutex>
#include <string>
#include <unordered_map>

#include "pcl_internal.h"
#include "pcl_ptx.cuh"

namespace pcl {

namespace {

constexpr int kTileM = 128;
constexpr int kBlockC = 32;                      // fp32 elements per 128-byte swizzle row
constexpr int kABytes = kTileM * kBlockC * 4;    // 16 KB
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 224 * 1024;
constexpr int kEpiWarps = 8;                    // two per TMEM lane quarter, splitting the column chunks
constexpr int kEpiStageBytes = kEpiWarps * 4096;
constexpr int kSecondIssuerWarp = 2 + kEpiWarps;        // warp 10
constexpr int kThreads = (3 + kEpiWarps) * 32;
// Launches whose tiles have a short reduction (the few-channel first layer: three k-steps) are bound by the
// epilogue warps, each of which issues an instruction every ~7 cycles: those run sixteen of them (four per TMEM
// lane quarter, warps 11-18 added behind the second issuer's warp) under a 104-register cap.
constexpr int kEpiWarpsWide = 16;
constexpr int kThreadsWide = (3 + kEpiWarpsWide) * 32;
constexpr int kEpiStageBytesWide = kEpiWarpsWide * (4096 + 128);      // staging tiles, then one 32-float bias slot per warp

struct FpropParams {
    int bw_log2, bh_log2;       // box of output pixels: bw x bh x (128 / (bw*bh))
    int tiles_q, tiles_p, tiles_n, tiles_k;
    int BN;                     // output maps per tile, multiple of 32, <= 256
    int R, S, pad_h, pad_w, cblocks;
    int stride_h, stride_w, dil_w;      // convolution strides; pixels between consecutive taps of a kernel row
    long long o_sw, o_sh, o_sn;         // element strides of `out` / `mask_src` between adjacent q, p, n
    int N, P, Q, Kout;
    int act;
    int stages;
    int KS;                     // k-steps (plain: {A,B} pairs; halo: weight tiles of consecutive taps) per pipeline slot
    int bmn;                    // B (weights) is MN-major: laid out [Cin][R*S][Kout], read through {32 maps, reduction rows,
                                // tap, 32-map group} boxes with the 32-byte-atom swizzle (backward-data without a transposed copy)
    int flip;                   // tap t reads tap R*S-1-t of the weights
    int split_acc;              // two issuers with an accumulator each (2 x 2 x MT x BN TMEM columns)
    int issuers;                // MMA-issuing threads (1 or 2; see the kernel)
    int grp;                    // plain tiling: a slot's KS k-steps are KS consecutive channel blocks of one tap, fetched by
                                // ONE copy of A and one of B (slot layout: KS A tiles, then KS B tiles)
    int tmem_cols;
    int tw, th, tn;             // pixels a tile spans in q, p, n (= the box, or 2 x the box in one direction when MT = 2)
    // Halo mode (R*S > 1): the A operand of ALL taps of a channel block comes from one haloed input patch
    // of (th + R - 1) x (tw + S - 1) pixels, loaded once; a tap is a row-shifted view of it.  A tile is MT
    // (1 or 2) boxes of 8 x 16 pixels that share every weight tile.
    int halo, MT;
    int PW;                     // patch width in pixels
    int patch_bytes, a_buf_bytes, NA;
    int half_off_bytes;         // offset of the second box inside the patch
    int half_dq, half_dp;       // pixel offset of the second box inside the tile
    const float* bias;
    const float* mask_src;
    int mask_mode;              // what mask_src does to the output: 0 zero where mask_src <= 0 (ReLU gradient),
                                // 1 multiply by mask_src * (1 - mask_src) (sigmoid gradient, mask_src being the sigmoid's output),
                                // 2 out = mask_src - lr * output (the SGD update of a weight gradient; out may be mask_src)
    float lr;
    float* out;
    int tma_store;              // the epilogue writes `out` with TMA stores from the staging tiles (tmOut is valid)
    // Split reduction (few tiles, long reduction: the FC layers at small minibatch): ksplit > 1 cuts the k-steps of
    // every tile into ksplit equal ranges of kps k-steps, each a tile of its own whose raw accumulators go to
    // out + split * split_stride (the caller adds the splits, then bias and activation).  Plain tiling only.
    int ksplit, kps;
    size_t split_stride;
    // resident_b (haloed tiling, one k tile, few taps): the CTA's weight tiles are loaded once and stay in the ring
    // for every tile.
    int resident_b;
    // K = 8 slices of a 32-element channel block that hold anything but zeros (4 unless the few-channel path packs
    // fewer live taps x channels into a block: the MMAs of all-zero slices are not issued)
    int kslices;
    int colsum_cta;         // column sums are kept per CTA over all its tiles (tiles_k == 1) and written once, one row
                            // per (CTA, box, lane quarter), instead of one row per (tile, box, lane quarter)
    int tile_duo;           // two issuing threads, alternate tiles (resident weights, one patch per tile, even NA)
    int bias_in_smem;           // the CTA keeps bias[0 .. BN) in shared memory (tiles_k == 1: every tile has the same columns)
    unsigned char* pool_idx;    // optional, with pool_out: per pooled element the position of the maximum (bits 0-1) and bit 2
                                // if that maximum is <= 0
    float* pool_out;            // optional [N][P/2][Q/2][Kout]: 2x2 window maxima of the output
    float* colsum_rows;         // optional [m_tiles * MT * 4][Kout] per-(box, quarter) column sums of the output
    int inject_short_copy;      // test mode: the first slot is armed for 16 bytes more than are copied, so that the
                                // waits on it run out (exercises the give-up path; single-CTA launches only)
    unsigned int* status;       // device status word (status[1]: limit of the bounded waits in microseconds)
};

// Walks the persistent tile sequence t = blockIdx.x, blockIdx.x + gridDim.x, ... and keeps the tile's
// coordinates (k tile, q tile, p tile, n tile) in mixed-radix counters, so that no role pays integer
// divisions per tile.
struct TileIter {
    int t, kt, qi, pi, ni, sp;      // sp: reduction split (outermost; 0 unless ksplit > 1)
    int step, dk, dq, dp, dn, ds;
    __device__ void init(const FpropParams& p, int first, int stride) {
        t = first; step = stride;
        int m = first;
        kt = m % p.tiles_k; m /= p.tiles_k;
        qi = m % p.tiles_q; m /= p.tiles_q;
        pi = m % p.tiles_p; m /= p.tiles_p;
        ni = m % p.tiles_n; sp = m / p.tiles_n;
        m = stride;
        dk = m % p.tiles_k; m /= p.tiles_k;
        dq = m % p.tiles_q; m /= p.tiles_q;
        dp = m % p.tiles_p; m /= p.tiles_p;
        dn = m % p.tiles_n; ds = m / p.tiles_n;
    }
    __device__ void next(const FpropParams& p) {
        t += step;
        kt += dk; int c = kt >= p.tiles_k; kt -= c ? p.tiles_k : 0;
        qi += dq + c; c = qi >= p.tiles_q; qi -= c ? p.tiles_q : 0;
        pi += dp + c; c = pi >= p.tiles_p; pi -= c ? p.tiles_p : 0;
        ni += dn + c; c = ni >= p.tiles_n; ni -= c ? p.tiles_n : 0;
        sp += ds + c;
    }
};

// Two MMA issuers take turns: the thread that owns slot `seq` spins (bounded) until the slots before it have
// been issued.  The other thread is at most one slot of MMAs away, so the wait is short.
__device__ __forceinline__ bool wait_issue_turn(volatile uint32_t* issue_seq, uint32_t seq, volatile uint32_t* abort_flag,
                                                unsigned int* status_word) {
    if (*issue_seq == seq) return true;
    unsigned long long t0 = 0, limit = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (*issue_seq == seq) return true;
        if ((spin & 255u) == 255u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_nanos();
            if (t0 == 0) { t0 = now; limit = wait_limit_nanos(status_word); }
            else if (now - t0 > limit) break;
        }
    }
    *abort_flag = 1u;
    atomicCAS(status_word, 0u, static_cast<unsigned int>(WAIT_ISSUE_TURN));
    return false;
}

// What the issuing thread needs from the kernel body.
struct IssuerCtx {
    uint8_t* smem;
    uint8_t* b_ring;
    uint64_t *full_bar, *empty_bar, *fullA_bar, *emptyA_bar, *tmem_full_bar, *tmem_empty_bar;
    volatile uint32_t* abort_flag;
    volatile uint32_t* issue_seq;
    uint32_t tmem_base, b_bytes, step_bytes, stage_bytes;
    int first_tile, tile_stride, total_tiles, kiters;
};

// 2x2 pooling of four channels: running maximum and its position e (0..3, row-major in the window; the FIRST
// maximum wins, as in the pooling kernels), one position per channel in the bytes of `arg`.
__device__ __forceinline__ void pool_take(float4& m, uint32_t& arg, const float4 t, const uint32_t e) {
    if (t.x > m.x) { m.x = t.x; arg = (arg & 0xffffff00u) | e; }
    if (t.y > m.y) { m.y = t.y; arg = (arg & 0xffff00ffu) | (e << 8); }
    if (t.z > m.z) { m.z = t.z; arg = (arg & 0xff00ffffu) | (e << 16); }
    if (t.w > m.w) { m.w = t.w; arg = (arg & 0x00ffffffu) | (e << 24); }
}
// position bytes plus bit 2 where the maximum is not positive (what a ReLU mask on the pooled layer would zero)
__device__ __forceinline__ uint32_t pool_code(const float4 m, const uint32_t arg) {
    return arg | (m.x > 0.f ? 0u : 4u) | (m.y > 0.f ? 0u : 4u << 8) | (m.z > 0.f ? 0u : 4u << 16) | (m.w > 0.f ? 0u : 4u << 24);
}
__device__ __forceinline__ float4 finish4(float4 o, const float4 b, const int act) {
    o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
    if (act == PCL_ACT_RELU) {
        o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
    } else if (act == PCL_ACT_SIGMOID) {
        o.x = sigmoid_fast(o.x); o.y = sigmoid_fast(o.y);
        o.z = sigmoid_fast(o.z); o.w = sigmoid_fast(o.w);
    }
    return o;
}

// v += the 32 x 32 block at `taddr` (the second issuer's accumulator).
__device__ __forceinline__ void add_second_accumulator(uint32_t taddr, uint32_t (&v)[32]) {
    uint32_t w[32];
    tmem_ld_32x32(taddr, w);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + __uint_as_float(w[i]));
}

// kTaps consecutive taps of a haloed slot, straight-line (the issuing role is a chain of dependent instructions: a taken
// branch costs it tens of cycles).
// kNsl = 0: the number of K = 8 slices per tap is the run-time `nsl` (skipped slices still cost their issue slots);
// kNsl = 1..3: exactly that many MMAs per tap are emitted (few-channel layers, whose tap rows hold fewer than 32
// live reduction elements: the issuing thread, not the tensor pipe, is what bounds their tiles).
template <bool kPair, int kTaps, int kMT, int kNsl = 0>
__device__ __forceinline__ void halo_taps(uint32_t d_tmem, uint32_t BN, uint32_t& a_lo, uint32_t b_lo, int& s, int S,
                                          uint32_t row16, uint32_t half_off16, uint32_t b16, uint32_t a_hi,
                                          uint32_t b_hi, uint32_t idesc, uint32_t& accum, uint32_t bks, uint32_t nsl) {
#pragma unroll
    for (int j = 0; j < kTaps; ++j) {
        if constexpr (kNsl == 0) {
            umma_kstep_tf32_bs<kPair>(d_tmem, a_lo, b_lo, a_hi, b_hi, idesc, accum, bks, nsl);
            if (kMT == 2) umma_kstep_tf32_bs<kPair>(d_tmem + BN, a_lo + half_off16, b_lo, a_hi, b_hi, idesc, accum, bks, nsl);
        } else {
#pragma unroll
            for (int h = 0; h < kMT; ++h) {
#pragma unroll
                for (int k = 0; k < kNsl; ++k) {
                    const uint64_t da = (uint64_t(a_hi) << 32) | (a_lo + (h ? half_off16 : 0u) + 2u * k);
                    const uint64_t db = (uint64_t(b_hi) << 32) | (b_lo + bks * k);
                    if constexpr (kPair) umma_tf32_pair(d_tmem + (h ? BN : 0u), da, db, idesc, k == 0 ? accum : 1u);
                    else umma_tf32(d_tmem + (h ? BN : 0u), da, db, idesc, k == 0 ? accum : 1u);
                }
            }
        }
        accum = 1;
        b_lo += b16;
        const bool wrap = ++s == S;     // the tap (r, s): next pixel of the patch, or the start of the next patch row
        a_lo += wrap ? 8 + row16 : 8;
        s = wrap ? 0 : s;
    }
}

// The MMA-issuing role, one warp per issuer (waits included), kept out of line and free of anything the loops do not
// need.  The WHOLE warp runs it, every lane with the same values, and the MMA and commit forms elect one lane to issue:
// run by lane 0 alone the same loops are divergent code whose descriptors the compiler moves into uniform registers
// word by word, at twice the cycles per MMA.  Even so a barrier poll or a commit costs the role ~80 cycles, so per
// slot it spends a few hundred cycles outside the MMAs, which the MMA queue (~4 deep) hides only behind wide MMAs
// (N = 256).  kDuo: two issuers take the slots alternately, so that one's bookkeeping overlaps the other's MMAs.  MMAs of both accumulate into the same tile (the pipe executes them one
// after another whichever thread issued them); a sequence number in shared memory makes the threads issue slot g
// only after slot g-1 has been issued, so the order of the additions, and with it every bit of the result, is
// that of a single issuer.
template <bool kPair, bool kDuo>
__device__ __noinline__ void mma_issuer(const FpropParams& p, const IssuerCtx& c, const uint32_t issuer) {
    // Everything the loops use is copied into registers first: the asm statements below clobber memory, so
    // anything left behind a reference would be re-read after each of them.
    const int BN = p.BN, KS = p.KS, MT = p.MT, NA = p.NA, PW = p.PW, S = p.S, taps = p.R * p.S;
    const int a_buf_bytes = p.a_buf_bytes, cblocks = p.cblocks, grp = p.grp, halo = p.halo, stages = p.stages;
    const uint32_t half_off16 = p.half_off_bytes >> 4;
    unsigned int* const status = p.status;
    volatile uint32_t* const abort_flag = c.abort_flag;
    volatile uint32_t* const issue_seq = c.issue_seq;
    uint8_t* const smem = c.smem;
    const uint32_t fullA0 = smem_u32(&c.fullA_bar[0]), emptyA0 = smem_u32(&c.emptyA_bar[0]);
    const uint32_t tfull0 = smem_u32(&c.tmem_full_bar[0]), tempty0 = smem_u32(&c.tmem_empty_bar[0]);
    const uint32_t tmem_base = c.tmem_base, b16 = c.b_bytes >> 4;
    const int first_tile = c.first_tile, tile_stride = c.tile_stride, total_tiles = c.total_tiles, kiters = c.kiters;

    // kDuo with `split`: each issuer accumulates its slots into an accumulator of its own (the epilogue adds the
    // two), so no ordering between the threads' MMAs can change a bit of the result and a thread passes the turn on
    // as soon as it has its slot, before issuing.  The slot STARTS stay ordered: letting one issuer overtake the
    // other (no turn at all) gave, rarely, wrong sums and lost slot releases on a 96-wide plain tiling with three
    // stages; cause not found, ordered starts are clean (40 x 40 repetitions, bit-identical).
    const bool split = kDuo && p.split_acc;
    const bool resident = p.resident_b != 0;
    const uint32_t nsl = uint32_t(p.kslices);      // (single issuer, haloed tiling: every tile reads the same weight slots)
    const int bmn = p.bmn;
    const uint32_t idesc = make_idesc_tf32(BN, false, bmn != 0, kPair ? 256u : 128u);
    const uint32_t bks = bmn ? 64u : 2u;         // k-block stride of B inside a k-step (16-byte units)
    // Descriptors differ only in the 14-bit address field (address >> 4) of their low word: the loops keep low
    // words in registers and advance them by addition.
    // The ring descriptor is B's in the haloed tiling (the ring holds weight tiles only) and A's in the plain one
    // (B's low word is then A's plus an offset that also carries the difference of the leading-offset fields).
    // MN-major B: 32-map groups are `b_group` bytes apart, 4-row reduction groups 512.
    const uint32_t b_group = (!halo && grp) ? KS * 4096u : 4096u;
    const uint64_t k_desc0 = make_smem_desc(smem_u32(halo ? c.b_ring : smem), 16, 1024, kSwizzle128B);
    const uint64_t m_desc0 = make_smem_desc(smem_u32(halo ? c.b_ring : smem), b_group, 512, kSwizzle128B_Atom32B);
    const uint32_t a_hi_plain = uint32_t(k_desc0 >> 32);
    const uint32_t b_hi = uint32_t((bmn ? m_desc0 : k_desc0) >> 32);
    const uint32_t ring_lo0 = uint32_t((halo && bmn) ? m_desc0 : k_desc0);
    const uint32_t b_lbo_delta = bmn ? uint32_t(m_desc0) - uint32_t(k_desc0) : 0u;
    const uint32_t full0 = smem_u32(&c.full_bar[0]), empty0 = smem_u32(&c.empty_bar[0]);
    const uint32_t stage16 = c.stage_bytes >> 4, step16 = c.step_bytes >> 4;
    // where k-step j of a slot finds its operands (16-byte units from the slot start)
    const uint32_t a_step16 = grp ? (kABytes >> 4) : step16;
    const uint32_t b_off16 = (grp ? KS * (kABytes >> 4) : (kABytes >> 4)) + b_lbo_delta;
    const uint32_t b_step16 = grp ? (bmn ? 256u : b16) : step16;

    uint32_t full_a = full0, empty_a = empty0, slot_lo = ring_lo0;     // ring position
    int stage = 0;
    uint32_t phase = 0;
    uint32_t turn = 0, seq = 0;     // kDuo: whose slot comes next; slots so far (both threads count alike)
    // tile_duo: the two issuing threads take the CTA's tiles alternately, each with its own accumulator set and its
    // own patch buffers (NA is even), so nothing orders them against each other; the weights stay resident.
    const bool leader = elected_lane();       // the lane that issues; it alone publishes the turn
    const bool tduo = !kDuo && p.tile_duo != 0;
    const int cnt0 = tduo ? int(issuer) : 0, cnt_step = tduo ? 2 : 1;
    int a_slot = cnt0;
    uint32_t phaseA = 0;
    int tile_cnt = cnt0;
    bool ok = true;

#define PCL_SLOT_BEGIN()                                                                                          \
    bool mine = true;                                                                                             \
    if (kDuo) { mine = turn == issuer; turn ^= 1u; }
#define PCL_SLOT_ACQUIRE()                                                                                        \
    if (!(resident && tile_cnt > cnt0) &&                                                                         \
        !bounded_wait_addr_warp(full_a, phase, abort_flag, status, WAIT_MMA_FULL)) { ok = false; break; }        \
    if (kDuo && !__all_sync(0xffffffffu, wait_issue_turn(issue_seq, seq, abort_flag, status))) { ok = false; break; } \
    if (kDuo && split && leader) *issue_seq = seq + 1;     /* split: only the slot STARTS are ordered (see below) */ \
    __syncwarp();                                                                                                 \
    tc_fence_after();
#define PCL_SLOT_RELEASE()                                                                                        \
    /* ordered hand-over: this thread's MMAs are fenced before the turn is published (the other issuer fences  */ \
    /* after reading it), so that MMAs of consecutive slots into one accumulator are ordered across the threads */ \
    if (kDuo && !split) { tc_fence_before(); if (leader) *issue_seq = seq + 1; __syncwarp(); }                    \
    if (!resident) umma_commit_addr<kPair>(empty_a);
#define PCL_SLOT_END()                                                                                            \
    if (kDuo) ++seq;                                                                                              \
    if (!split || mine) accum = 1;      /* split: an issuer's own first slot overwrites its own accumulator */    \
    full_a += 8; empty_a += 8; slot_lo += stage16;                                                                \
    if (++stage == stages) { stage = 0; phase ^= 1u; full_a = full0; empty_a = empty0; slot_lo = ring_lo0; }

    for (int t = first_tile + cnt0 * tile_stride; t < total_tiles && ok; t += cnt_step * tile_stride, tile_cnt += cnt_step) {
        const uint32_t acc = tile_cnt & 1;
        const uint32_t acc_phase = (tile_cnt >> 1) & 1;
        if (!bounded_wait_addr_warp(tempty0 + acc * 8, acc_phase ^ 1u, abort_flag, status, WAIT_MMA_TMEM_EMPTY)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (split ? (2 * acc + issuer) * MT * BN : acc * MT * BN);
        uint32_t accum = 0;         // the tile's first MMA (whoever issues it) overwrites the accumulator
        if (resident) { stage = 0; phase = 0; full_a = full0; empty_a = empty0; slot_lo = ring_lo0; }
        if (halo) {
            const uint64_t a_desc0 = make_smem_desc(0, 16, PW * 128, kSwizzle128B);   // 8-pixel groups are one patch row apart
            const uint32_t a_hi = uint32_t(a_desc0 >> 32);
            const uint32_t row16 = (PW - S) * 8;        // from the end of a tap row to the start of the next
            for (int cb = 0; cb < cblocks && ok; ++cb) {
                if (!bounded_wait_addr_warp(fullA0 + a_slot * 8, phaseA, abort_flag, status, WAIT_MMA_FULL)) { ok = false; break; }
                // the tap (r, s) = a shift by (r * PW + s) pixels of 128 bytes inside the patch
                uint32_t a_lo = uint32_t(a_desc0) + ((smem_u32(smem + a_slot * a_buf_bytes) & 0x3FFFFu) >> 4);
                int s = 0;
                for (int tap = 0; tap < taps; tap += KS) {
                    const int nst = taps - tap < KS ? taps - tap : KS;
                    PCL_SLOT_BEGIN()
                    if (mine) {
                        PCL_SLOT_ACQUIRE()
                        if (MT == 2) {
                            if (nst == 3 && nsl == 2) halo_taps<kPair, 3, 2, 2>(d_tmem, BN, a_lo, slot_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            else if (nst == 3) halo_taps<kPair, 3, 2>(d_tmem, BN, a_lo, slot_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            else if (nst == 2) halo_taps<kPair, 2, 2>(d_tmem, BN, a_lo, slot_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            else {
                                uint32_t b_lo = slot_lo;
                                for (int j = 0; j < nst; ++j, b_lo += b16)
                                    halo_taps<kPair, 1, 2>(d_tmem, BN, a_lo, b_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            }
                        } else {
                            if (nst == 3) halo_taps<kPair, 3, 1>(d_tmem, BN, a_lo, slot_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            else if (nst == 2) halo_taps<kPair, 2, 1>(d_tmem, BN, a_lo, slot_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            else {
                                uint32_t b_lo = slot_lo;
                                for (int j = 0; j < nst; ++j, b_lo += b16)
                                    halo_taps<kPair, 1, 1>(d_tmem, BN, a_lo, b_lo, s, S, row16, half_off16, b16, a_hi, b_hi, idesc, accum, bks, nsl);
                            }
                        }
                        PCL_SLOT_RELEASE()
                    } else {
                        for (int j = 0; j < nst; ++j) {
                            const bool wrap = ++s == S;
                            a_lo += wrap ? 8 + row16 : 8;
                            s = wrap ? 0 : s;
                        }
                    }
                    PCL_SLOT_END()
                }
                if (ok) umma_commit_addr<kPair>(emptyA0 + a_slot * 8);       // one arrival per issuer
                a_slot += cnt_step;
                if (a_slot >= NA) { a_slot -= NA; phaseA ^= 1u; }
            }
        } else if (KS == 2 && grp) {
            // two k-steps per slot, fetched by one copy per operand (the hot loop of the wide layers)
            for (int kit = 0; kit < kiters; kit += 2) {
                PCL_SLOT_BEGIN()
                if (mine) {
                    PCL_SLOT_ACQUIRE()
                    umma_kstep_tf32_bs<kPair>(d_tmem, slot_lo, slot_lo + b_off16, a_hi_plain, b_hi, idesc, accum, bks, nsl);
                    umma_kstep_tf32_bs<kPair>(d_tmem, slot_lo + a_step16, slot_lo + b_off16 + b_step16, a_hi_plain, b_hi, idesc, 1, bks, nsl);
                    PCL_SLOT_RELEASE()
                }
                PCL_SLOT_END()
            }
        } else {
            for (int kit = 0; kit < kiters; kit += KS) {
                const int nst = kiters - kit < KS ? kiters - kit : KS;
                PCL_SLOT_BEGIN()
                if (mine) {
                    PCL_SLOT_ACQUIRE()
                    uint32_t a_lo = slot_lo, b_lo = slot_lo + b_off16;
                    for (int j = 0; j < nst; ++j, a_lo += a_step16, b_lo += b_step16) {
                        umma_kstep_tf32_bs<kPair>(d_tmem, a_lo, b_lo, a_hi_plain, b_hi, idesc, accum, bks, nsl);
                        accum = 1;
                    }
                    PCL_SLOT_RELEASE()
                }
                PCL_SLOT_END()
            }
        }
        if (ok) umma_commit_addr<kPair>(tfull0 + acc * 8);       // one arrival per issuer
    }
#undef PCL_SLOT_BEGIN
#undef PCL_SLOT_ACQUIRE
#undef PCL_SLOT_RELEASE
#undef PCL_SLOT_END
}

// kPair: two CTAs of a cluster (ranks 0 and 1) compute two M tiles (consecutive image groups) against the
// same BN = 256 weight tile with M = 256 MMAs issued by rank 0; each CTA loads its own A tile and only half
// of the weight rows, which cuts the shared-memory fill traffic per MMA by a third (plain tiling only).
// kPool: the epilogue also writes the 2x2 window maxima (kept out of the other instantiations, whose epilogue it
// would cost registers).
// kMask: the epilogue applies the ReLU mask (backward-data); its eight prefetched mask vectors would cost the other
// instantiations registers (the epilogue is what the 168-register budget of an 11-warp CTA is short of, and a
// spilled value that has left L1 costs ~600 cycles per use).
template <bool kPair, bool kPool, bool kMask, int kEpi = kEpiWarps>
__global__ void __launch_bounds__((3 + kEpi) * 32, 1)
tc_fprop_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ FpropParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages];
    __shared__ uint64_t empty_bar[kMaxStages];
    __shared__ uint64_t fullA_bar[4];
    __shared__ uint64_t emptyA_bar[4];
    __shared__ uint64_t tmem_full_bar[2];
    __shared__ uint64_t tmem_empty_bar[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_flag;
    __shared__ volatile uint32_t issue_seq;      // two issuers: number of slots whose MMAs have been issued
    __shared__ __align__(16) float bias_s[256];  // the tile's bias values (launches whose tiles all have the same columns)

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // plain mode: ring of {A 16 KB, B BN*128 B} slots.  halo mode: NA patch buffers, then a ring of B slots.
    // A slot holds KS k-steps: the issuing thread pays one barrier round trip and one commit per slot, which
    // is what bounds narrow tiles (their MMAs are short), so narrow tiles batch several k-steps per slot.
    const uint32_t b_bytes = kPair ? p.BN * 64 : p.BN * 128;
    const uint32_t pair_rank = kPair ? cluster_ctarank() : 0u;
    const int first_tile = kPair ? int(cluster_id_x()) : int(blockIdx.x);
    const int tile_stride = kPair ? int(nclusters_x()) : int(gridDim.x);
    const uint32_t step_bytes = p.halo ? b_bytes : kABytes + b_bytes;
    const uint32_t stage_bytes = p.KS * step_bytes;
    uint8_t* b_ring = smem + (p.halo ? p.NA * p.a_buf_bytes : kABytes);
    uint8_t* epi_stage = smem + (p.halo ? p.NA * p.a_buf_bytes : 0) + p.stages * stage_bytes;   // kEpi x 4 KB (+ kEpi x 128 B of bias slots in the 16-warp variant)

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 4; ++a) {
            mbar_init(&fullA_bar[a], 1);
            mbar_init(&emptyA_bar[a], p.issuers);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&tmem_full_bar[a], p.issuers);
            mbar_init(&tmem_empty_bar[a], kPair ? 2 * kEpi : kEpi);
        }
        abort_flag = 0;
        issue_seq = 0;
        mbar_fence_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        if constexpr (kPair) { tmem_alloc_pair(&tmem_base_slot, p.tmem_cols); tmem_relinquish_pair(); }
        else { tmem_alloc(&tmem_base_slot, p.tmem_cols); tmem_relinquish(); }
    }
    if (kPool && p.bias_in_smem)
        for (int i = threadIdx.x; i < 256; i += blockDim.x) bias_s[i] = (p.bias && i < p.Kout) ? __ldg(p.bias + i) : 0.f;
    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync_all();     // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2;
    const int m_tiles = p.tiles_q * p.tiles_p * p.tiles_n;
    const int total_tiles = m_tiles * p.tiles_k * p.ksplit;
    const int kiters = p.ksplit > 1 ? p.kps : p.R * p.S * p.cblocks;       // k-steps of one tile

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // The whole warp runs the loop (every lane the same values) and an elected lane issues the copies and arms the
        // barriers; the loop is kept to a few instructions per copy (addresses and coordinates advance by addition).
        {
            int stage = 0, issued = 0;
            uint32_t phase = 0;
            int a_slot = 0, issuedA = 0;
            uint32_t phaseA = 0;
            bool ok = true;
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            const uint32_t ring0 = smem_u32(p.halo ? b_ring : smem);
            uint32_t full_a = full0, empty_a = empty0, slot_a = ring0;
            const uint32_t full_dst0 = kPair ? map_to_cta(&full_bar[0], 0) : full0;   // where the copies complete
            uint32_t full_dst = full_dst0;
            const int c_end = p.cblocks * kBlockC;
            const int taps = p.R * p.S;
            TileIter it;
            for (it.init(p, first_tile, tile_stride); it.t < total_tiles && ok; it.next(p)) {
                const int q0 = it.qi * p.tw, p0 = it.pi * p.th;
                const int n0 = (kPair ? 2 * it.ni + int(pair_rank) : it.ni) * p.tn;
                const int kcol = it.kt * p.BN + (kPair ? int(pair_rank) * (p.BN >> 1) : 0);
                if (p.halo) {
                    for (int c0 = 0; c0 < c_end && ok; c0 += kBlockC) {
                        if (!bounded_wait_warp(&emptyA_bar[a_slot], phaseA ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) {
                            ok = false;
                            break;
                        }
                        if (!kPair) mbar_expect_tx(&fullA_bar[a_slot], p.patch_bytes);
                        else if (pair_rank == 0) mbar_expect_tx(&fullA_bar[a_slot], 2 * p.patch_bytes);
                        tma_load_4d_addr<kPair>(smem_u32(smem + a_slot * p.a_buf_bytes), &tmA,
                                                kPair ? map_to_cta(&fullA_bar[a_slot], 0) : smem_u32(&fullA_bar[a_slot]),
                                                c0, q0 - p.pad_w, p0 - p.pad_h, n0);
                        ++issuedA;
                        if (++a_slot == p.NA) { a_slot = 0; phaseA ^= 1u; }
                        for (int tap = 0; tap < taps; tap += p.KS) {
                            if (p.resident_b && it.t != first_tile) break;      // (loaded for the first tile, never released)
                            if (!bounded_wait_addr_warp(empty_a, phase ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) {
                                ok = false;
                                break;
                            }
                            const int nst = taps - tap < p.KS ? taps - tap : p.KS;
                            const int ncp = p.grp ? p.KS : nst;       // a box counts in full, also where it is filled with zeros
                            if (!kPair) mbar_expect_tx_addr(full_a, ncp * b_bytes);
                            else if (pair_rank == 0) mbar_expect_tx_addr(full_a, 2 * ncp * b_bytes);
                            if (p.grp) {
                                // the slot's taps in one copy (box {32 channels, BN maps, KS taps}; taps past the last
                                // one are outside the tensor: filled with zeros and not used)
                                tma_load_3d_addr<kPair>(slot_a, &tmB, full_dst, c0, kcol, tap);
                            } else {
                                uint32_t dst = slot_a;
                                for (int j = 0; j < nst; ++j, dst += b_bytes)
                                    if (p.bmn) tma_load_4d_addr<kPair>(dst, &tmB, full_dst, 0, c0, p.flip ? taps - 1 - (tap + j) : tap + j, kcol >> 5);
                                    else tma_load_3d_addr<kPair>(dst, &tmB, full_dst, c0, tap + j, kcol);
                            }
                            ++issued;
                            full_a += 8; empty_a += 8; full_dst += 8; slot_a += stage_bytes;
                            if (++stage == p.stages) {
                                stage = 0; phase ^= 1u;
                                full_a = full0; empty_a = empty0; full_dst = full_dst0; slot_a = ring0;
                            }
                        }
                    }
                } else {
                    // k-step order: r, then s, then channel block; a reduction split starts kps k-steps further
                    int c0 = 0, s = 0, tap = 0;
                    // (input coordinates of the tile's first pixel for tap (0, 0); a strided layer's box takes every
                    // stride-th pixel from there)
                    int cq = q0 * p.stride_w - p.pad_w, cp = p0 * p.stride_h - p.pad_h;
                    const int dil = p.dil_w, row_back = p.S * p.dil_w;
                    if (p.ksplit > 1) {
                        const int kit0 = it.sp * kiters;
                        tap = kit0 / p.cblocks;
                        c0 = (kit0 - tap * p.cblocks) * kBlockC;
                        const int r0 = tap / p.S;
                        s = tap - r0 * p.S;
                        cq += s * dil; cp += r0;
                    }
                    for (int kit = 0; kit < kiters; kit += p.KS) {
                        if (!bounded_wait_addr_warp(empty_a, phase ^ 1u, &abort_flag, p.status, WAIT_PRODUCER_EMPTY)) {
                            ok = false;
                            break;
                        }
                        const int nst = kiters - kit < p.KS ? kiters - kit : p.KS;
                        // pair: both CTAs' copies complete on the leader's barrier, which its producer arms
                        if (!kPair) mbar_expect_tx_addr(full_a, nst * step_bytes + (p.inject_short_copy && issued == 0 ? 16 : 0));
                        else if (pair_rank == 0) mbar_expect_tx_addr(full_a, 2 * nst * step_bytes);
                        uint32_t dst = slot_a;
                        if (p.grp) {
                            // (cblocks is a multiple of KS here, so nst = KS and a slot never straddles two taps)
                            tma_load_5d_addr<kPair>(dst, &tmA, full_dst, 0, cq, cp, n0, c0 >> 5);
                            if (p.bmn) tma_load_4d_addr<kPair>(dst + p.KS * kABytes, &tmB, full_dst, 0, c0, p.flip ? taps - 1 - tap : tap, kcol >> 5);
                            else tma_load_4d_addr<kPair>(dst + p.KS * kABytes, &tmB, full_dst, 0, kcol, c0 >> 5, tap);
                            c0 += p.KS * kBlockC;
                            if (c0 == c_end) {
                                c0 = 0; ++tap; cq += dil;
                                if (++s == p.S) { s = 0; cq -= row_back; ++cp; }
                            }
                        } else
                        for (int j = 0; j < nst; ++j, dst += step_bytes) {
                            tma_load_4d_addr<kPair>(dst, &tmA, full_dst, c0, cq, cp, n0);
                            if (p.bmn) tma_load_4d_addr<kPair>(dst + kABytes, &tmB, full_dst, 0, c0, p.flip ? taps - 1 - tap : tap, kcol >> 5);
                            else tma_load_3d_addr<kPair>(dst + kABytes, &tmB, full_dst, c0, tap, kcol);
                            c0 += kBlockC;
                            if (c0 == c_end) {
                                c0 = 0; ++tap; cq += dil;
                                if (++s == p.S) { s = 0; cq -= row_back; ++cp; }
                            }
                        }
                        ++issued;
                        full_a += 8; empty_a += 8; full_dst += 8; slot_a += stage_bytes;
                        if (++stage == p.stages) {
                            stage = 0; phase ^= 1u;
                            full_a = full0; empty_a = empty0; full_dst = full_dst0; slot_a = ring0;
                        }
                    }
                }
            }
            if (!ok) {
                // Gave up: the copies already issued still land in this CTA's shared
                // memory, so wait (bounded) for each armed slot before leaving.
                int pending = issued < p.stages ? issued : p.stages;
                for (int j = 0; j < pending; ++j) {
                    if (--stage < 0) { stage = p.stages - 1; phase ^= 1u; }
                    for (uint32_t spin = 0; spin < (1u << 20); ++spin)
                        if (mbar_try_wait(&full_bar[stage], phase)) break;
                }
                pending = issuedA < p.NA ? issuedA : p.NA;
                for (int j = 0; j < pending; ++j) {
                    if (--a_slot < 0) { a_slot = p.NA - 1; phaseA ^= 1u; }
                    for (uint32_t spin = 0; spin < (1u << 20); ++spin)
                        if (mbar_try_wait(&fullA_bar[a_slot], phaseA)) break;
                }
            }
        }
    } else if (warp == 1 || warp == kSecondIssuerWarp) {
        // --------------------------------------------------------- MMA issuers
        const uint32_t issuer = warp == 1 ? 0u : 1u;
        if (pair_rank == 0 && issuer < uint32_t(p.tile_duo ? 2 : p.issuers)) {     // the whole warp (see mma_issuer)
            IssuerCtx c;
            c.smem = smem; c.b_ring = b_ring;
            c.full_bar = full_bar; c.empty_bar = empty_bar; c.fullA_bar = fullA_bar; c.emptyA_bar = emptyA_bar;
            c.tmem_full_bar = tmem_full_bar; c.tmem_empty_bar = tmem_empty_bar;
            c.abort_flag = &abort_flag; c.issue_seq = &issue_seq;
            c.tmem_base = tmem_base; c.b_bytes = b_bytes; c.step_bytes = step_bytes; c.stage_bytes = stage_bytes;
            c.first_tile = first_tile; c.tile_stride = tile_stride; c.total_tiles = total_tiles; c.kiters = kiters;
            if (p.issuers == 2) mma_issuer<kPair, true>(p, c, issuer);
            else mma_issuer<kPair, false>(p, c, issuer);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3;           // TMEM lanes 32*quarter .. +31
        const int epi = warp < kSecondIssuerWarp ? warp - 2 : warp - 3;     // 0 .. kEpi-1 (warp 10 is an issuer)
        // the quarter's kEpi/4 warps share its (box, 32-column chunk) items: warp `sub` takes every (kEpi/4)-th
        constexpr int kSub = kEpi / 4;
        const int sub = epi >> 2;               // (warps 2-5: 0, 6-9: 1, 11-14: 2, 15-18: 3; one of each per quarter)
        const int cpb = p.BN / 32;              // chunks per box
        const int row = quarter * 32 + lane;    // row of the tile = pixel of the box
        const int iw = row & (bw - 1);
        const int ih = (row >> p.bw_log2) & (bh - 1);
        const int in_ = row >> (p.bw_log2 + p.bh_log2);      // halo mode: the box is 8 x 16 x 1, so in_ = 0
        const bool vec_ok = (p.Kout & 3) == 0;
        int tile_cnt = 0;
        TileIter it;
        // per-CTA column sums (colsum_cta): this lane's partial sums of the warp's (at most four) chunks of a tile
        float4 cacc0 = make_float4(0.f, 0.f, 0.f, 0.f), cacc1 = cacc0, cacc2 = cacc0, cacc3 = cacc0;
        bool pooled_only = false;
        if constexpr (kPool) pooled_only = !p.out && p.act != PCL_ACT_SIGMOID && (kEpi > kEpiWarps || (!kMask && p.tma_store));
        if (pooled_only) {
            // Pooled output only (the step never reads the full-resolution output of a pooled layer).  The raw
            // accumulators are staged, each lane takes two windows of its four columns, adds the bias to the four
            // values s_e of a window, takes their maximum m and applies the activation to m alone: max commutes with
            // the (monotone) bias add and ReLU, so the stored maximum is bit for bit the maximum of the finished
            // values.  Position code: the first e with act(s_e) == act(m), i.e. with s_e == m, except that under ReLU a
            // window with m <= 0 holds four zeros, whose first maximum is e = 0.
            // Few-channel layers are bound by these warps, not by the tensor pipe: everything that does not depend on
            // the tile is computed once, a box without a chunk for this warp costs it nothing, and the accumulator set
            // is handed back as soon as the warp's last chunk is in registers.
            const int lb = p.bw_log2;
            const uint32_t stg = smem_u32(epi_stage + epi * 4096);
            const uint32_t my_row = stg + lane * 128, my_x = (lane & 7) * 16;
            const int P2 = p.P >> 1, Q2 = p.Q >> 1;
            uint32_t ld_a[2][4];
            int wdq[2], wdp[2], wdn[2];
            uint32_t woff[2];           // the window's pooled element inside the tile's pooled block (+ this lane's columns)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int wdx = (lane >> 3) + 4 * half;
                const int r0 = ((wdx & ((1 << (lb - 1)) - 1)) << 1) | ((wdx >> (lb - 1)) << (lb + 1));
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int rr = r0 | (e & 1) | ((e >> 1) << lb);
                    ld_a[half][e] = stg + rr * 128 + (((lane & 7) ^ (rr & 7)) * 16);
                }
                const int wrow = quarter * 32 + r0;
                wdq[half] = wrow & (bw - 1);
                wdp[half] = (wrow >> p.bw_log2) & (bh - 1);
                wdn[half] = wrow >> (p.bw_log2 + p.bh_log2);
                woff[half] = uint32_t(((wdn[half] * P2 + (wdp[half] >> 1)) * Q2 + (wdq[half] >> 1)) * p.Kout + (lane & 7) * 4);
            }
            int my_items = 0;           // chunks of a tile that are this warp's
            for (int h = 0; h < p.MT; ++h)
                for (int ch = (sub - h * cpb) & (kSub - 1); ch < cpb; ch += kSub) ++my_items;
            const bool relu = p.act == PCL_ACT_RELU;
            const uint32_t t_quarter = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const uint32_t t_second = p.MT * p.BN;      // split accumulators: the second issuer's copy of this box
            for (it.init(p, first_tile, tile_stride); it.t < total_tiles; it.next(p), ++tile_cnt) {
                const int acc = tile_cnt & 1;
                const int ni = kPair ? 2 * it.ni + int(pair_rank) : it.ni;
                const uint32_t acc_phase = (tile_cnt >> 1) & 1;
                if (!bounded_wait_warp(&tmem_full_bar[acc], acc_phase, &abort_flag, p.status, WAIT_EPI_TMEM_FULL)) break;
                tc_fence_after();
                int left = my_items;
                auto hand_back = [&]() {        // this warp has read all it needs of the accumulator set
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (kPair && pair_rank != 0) mbar_arrive_cluster(map_to_cta(&tmem_empty_bar[acc], 0));
                        else mbar_arrive(&tmem_empty_bar[acc]);
                    }
                };
                if (left == 0) hand_back();
                const int q_base = it.qi * p.tw, p_base = it.pi * p.th, n_base = ni * p.tn;
                for (int h = 0; h < p.MT; ++h) {
                    const int ch0 = (sub - h * cpb) & (kSub - 1);
                    if (ch0 >= cpb) continue;
                    const int qb = q_base + h * p.half_dq, pb = p_base + h * p.half_dp;
                    const size_t tile_off = ((static_cast<size_t>(n_base) * P2 + (pb >> 1)) * Q2 + (qb >> 1)) * p.Kout + it.kt * p.BN;
                    const bool w_ok[2] = {qb + wdq[0] < p.Q && pb + wdp[0] < p.P && n_base + wdn[0] < p.N,
                                          qb + wdq[1] < p.Q && pb + wdp[1] < p.P && n_base + wdn[1] < p.N};
                    const uint32_t t_row = t_quarter + ((p.split_acc ? 2 * acc : acc) * p.MT + h) * p.BN;
                    for (int ch = ch0; ch < cpb; ch += kSub) {
                        const int col = it.kt * p.BN + ch * 32 + (lane & 7) * 4;
                        float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (p.bias_in_smem) b = *reinterpret_cast<const float4*>(bias_s + ch * 32 + (lane & 7) * 4);
                        else if (p.bias && col < p.Kout) b = __ldg(reinterpret_cast<const float4*>(p.bias + col));
                        if constexpr (kEpi == kEpiWarps) {
                            uint32_t v[32];
                            tmem_ld_32x32(t_row + ch * 32, v);
                            tmem_ld_wait();
                            if (p.split_acc) add_second_accumulator(t_row + t_second + ch * 32, v);
                            if (--left == 0) hand_back();
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                st_shared_v4(my_row + ((j * 16) ^ my_x), __uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                             __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                        } else {
                            uint32_t v[16], u[16];
                            tmem_ld_32x16(t_row + ch * 32, v);
                            tmem_ld_32x16(t_row + ch * 32 + 16, u);
                            tmem_ld_wait();
                            if (--left == 0) hand_back();
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
                                st_shared_v4(my_row + ((jj * 16) ^ my_x), __uint_as_float(v[4 * jj]), __uint_as_float(v[4 * jj + 1]),
                                             __uint_as_float(v[4 * jj + 2]), __uint_as_float(v[4 * jj + 3]));
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
                                st_shared_v4(my_row + (((4 + jj) * 16) ^ my_x), __uint_as_float(u[4 * jj]), __uint_as_float(u[4 * jj + 1]),
                                             __uint_as_float(u[4 * jj + 2]), __uint_as_float(u[4 * jj + 3]));
                        }
                        __syncwarp();
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            float4 s0 = ld_shared_v4(ld_a[half][0]), s1 = ld_shared_v4(ld_a[half][1]);
                            float4 s2 = ld_shared_v4(ld_a[half][2]), s3 = ld_shared_v4(ld_a[half][3]);
                            auto one = [&](float a0, float a1, float a2, float a3, float bb, float& mo) -> uint32_t {
                                a0 += bb; a1 += bb; a2 += bb; a3 += bb;
                                const float m = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
                                uint32_t pos = a0 == m ? 0u : (a1 == m ? 1u : (a2 == m ? 2u : 3u));
                                const bool nonpos = !(m > 0.f);
                                if (relu) { mo = fmaxf(m, 0.f); pos = nonpos ? 0u : pos; } else { mo = m; }
                                return pos | (nonpos ? 4u : 0u);
                            };
                            float4 m;
                            const uint32_t c0 = one(s0.x, s1.x, s2.x, s3.x, b.x, m.x), c1 = one(s0.y, s1.y, s2.y, s3.y, b.y, m.y);
                            const uint32_t c2 = one(s0.z, s1.z, s2.z, s3.z, b.z, m.z), c3 = one(s0.w, s1.w, s2.w, s3.w, b.w, m.w);
                            if (w_ok[half] && col < p.Kout) {
                                const size_t po = tile_off + woff[half] + ch * 32;
                                *reinterpret_cast<float4*>(p.pool_out + po) = m;
                                if (p.pool_idx) *reinterpret_cast<uint32_t*>(p.pool_idx + po) = c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
                            }
                        }
                        __syncwarp();       // the staging tile is free for the next chunk
                    }
                }
            }
        } else
        for (it.init(p, first_tile, tile_stride); it.t < total_tiles; it.next(p), ++tile_cnt) {
            const int acc = tile_cnt & 1;
            const int ni = kPair ? 2 * it.ni + int(pair_rank) : it.ni;
            const uint32_t acc_phase = (tile_cnt >> 1) & 1;
            const int kt = it.kt;
            if (!bounded_wait_warp(&tmem_full_bar[acc], acc_phase, &abort_flag, p.status, WAIT_EPI_TMEM_FULL)) break;
            tc_fence_after();
            int cs_item = 0;        // running index of the warp's chunks in this tile (h-major), for the per-CTA sums
            for (int h = 0; h < p.MT; ++h) {
            const int ch0 = (sub - h * cpb) & (kSub - 1);       // first chunk of box h that is this warp's
            const int q = it.qi * p.tw + iw + h * p.half_dq;
            const int pp = it.pi * p.th + ih + h * p.half_dp;
            const int n = ni * p.tn + in_;
            const bool valid = (q < p.Q) && (pp < p.P) && (n < p.N);
            // element offset of the pixel's row in `out` (packed NPQK, or every stride-th pixel of a larger tensor)
            const size_t pix_off = static_cast<size_t>(n) * p.o_sn + static_cast<size_t>(pp) * p.o_sh + static_cast<size_t>(q) * p.o_sw;
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                   ((p.split_acc ? 2 * acc : acc) * p.MT + h) * p.BN;
            const uint32_t t_second = p.MT * p.BN;      // split accumulators: the second issuer's copy of this box
            float* cs_row = nullptr;
            if (p.colsum_rows && !p.colsum_cta && ni * p.tn < p.N) {      // (an odd image-group count leaves the pair's last tile empty)
                const size_t m_index = (static_cast<size_t>(ni) * p.tiles_p + it.pi) * p.tiles_q + it.qi;
                cs_row = p.colsum_rows + ((m_index * p.MT + h) * 4 + quarter) * p.Kout;
            }
            if (kEpi > kEpiWarps || (!kMask && p.tma_store)) {      // (wide-epilogue launches always stage)
                // TMA-store path (no mask, no column sums).  Each lane owns one row (pixel) of the accumulator: it
                // finishes its 32 columns in registers (bias, activation), puts them into its row of the warp's
                // 4 KB staging tile in the 128-byte-swizzle layout, and one lane hands the tile to TMA, which writes
                // the 32 pixels x 128 bytes and clips what lies outside the tensor.  The warp's 32 rows are 32
                // consecutive pixels of the box, i.e. a sub-box whose first pixel is (sq, sp, sn).
                const uint32_t stg = smem_u32(epi_stage + epi * 4096);
                const int srow = quarter * 32;
                for (int ch = ch0; ch < cpb; ch += kSub) {
                    const int col0 = kt * p.BN + ch * 32;
                    // (the 8-warp variant fetches the chunk's bias ahead of the accumulator, eight vectors per lane;
                    // under the 16-warp variant's register cap each lane fetches one value and the warp shares the
                    // 32 of them through 128 bytes of shared memory)
                    constexpr int kBv = kEpi > kEpiWarps ? 1 : 8;
                    float4 bv[kBv];
                    float bias_lane = 0.f;
                    if (kEpi == kEpiWarps) {
#pragma unroll
                        for (int j = 0; j < kBv; ++j)
                            bv[j] = (p.bias && col0 + 4 * j < p.Kout) ? __ldg(reinterpret_cast<const float4*>(p.bias + col0 + 4 * j))
                                                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                    } else {
                        // (the previous chunk's reads of the slot lie before the __syncwarp() that ended its staging)
                        if (p.bias && col0 + lane < p.Kout) bias_lane = __ldg(p.bias + col0 + lane);
                        reinterpret_cast<float*>(epi_stage + kEpi * 4096 + epi * 128)[lane] = bias_lane;
                    }
                    // finishes four columns (bias, activation) and puts them into the lane's row of the staging tile
                    auto finish_store = [&](const uint32_t* v4, const float4 bj, const int j) {
                        float4 o = make_float4(__uint_as_float(v4[0]) + bj.x, __uint_as_float(v4[1]) + bj.y,
                                               __uint_as_float(v4[2]) + bj.z, __uint_as_float(v4[3]) + bj.w);
                        if (p.act == PCL_ACT_RELU) {
                            o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
                        } else if (p.act == PCL_ACT_SIGMOID) {
                            o.x = sigmoid_fast(o.x); o.y = sigmoid_fast(o.y);
                            o.z = sigmoid_fast(o.z); o.w = sigmoid_fast(o.w);
                        }
                        st_shared_v4(stg + lane * 128 + ((j ^ (lane & 7)) * 16), o.x, o.y, o.z, o.w);
                    };
                    if constexpr (kEpi == kEpiWarps) {
                        uint32_t v[32];
                        tmem_ld_32x32(t_row + ch * 32, v);
                        tmem_ld_wait();
                        if (!kPool && p.split_acc) add_second_accumulator(t_row + t_second + ch * 32, v);
                        // the previous store of this warp must have read the staging tile before it is overwritten
                        if (lane == 0) bulk_wait_group_read0();
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j) finish_store(&v[4 * j], bv[j], j);
                    } else {
                        // two loads of 16 columns: half the registers
                        if (lane == 0) bulk_wait_group_read0();
                        __syncwarp();       // (also: every lane's bias value is in the warp's bias slot)
                        const uint32_t bias_a = smem_u32(epi_stage + kEpi * 4096 + epi * 128);    // behind the staging tiles
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            uint32_t v[16];
                            tmem_ld_32x16(t_row + ch * 32 + hh * 16, v);
                            tmem_ld_wait();
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
                                finish_store(&v[4 * jj], ld_shared_v4(bias_a + 16 * (hh * 4 + jj)), hh * 4 + jj);
                        }
                    }
                    fence_proxy_async_shared();
                    __syncwarp();
                    if (lane == 0 && col0 < p.Kout && p.out) {     // (pooling launches may keep y unstored)
                        const int sq = it.qi * p.tw + (srow & (bw - 1)) + h * p.half_dq;
                        const int sp = it.pi * p.th + ((srow >> p.bw_log2) & (bh - 1)) + h * p.half_dp;
                        const int sn = ni * p.tn + (srow >> (p.bw_log2 + p.bh_log2));
                        if (sq < p.Q && sp < p.P && sn < p.N) {     // (a store never starts outside the tensor)
                            tma_store_4d(&tmOut, stg, col0, sq, sp, sn);
                            bulk_commit_group();
                        }
                    }
                    if (kPool) {
                        // Fused 2x2 max pooling from the finished values in the staging tile: the 32 rows hold 8 whole
                        // windows (bit 0 of the row = parity of q, bit log2(bw) = parity of p; boxes start at even
                        // coordinates); lane l takes windows (l >> 3) and (l >> 3) + 4 of its 4 columns.
                        const int lb = p.bw_log2;
                        const int col = col0 + (lane & 7) * 4;
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const int wdx = (lane >> 3) + 4 * half;
                            const int r0 = ((wdx & ((1 << (lb - 1)) - 1)) << 1) | ((wdx >> (lb - 1)) << (lb + 1));
                            float4 m = ld_shared_v4(stg + r0 * 128 + (((lane & 7) ^ (r0 & 7)) * 16));
                            uint32_t arg = 0;
#pragma unroll
                            for (int e = 1; e < 4; ++e) {
                                const int rr = r0 | (e & 1) | ((e >> 1) << lb);
                                pool_take(m, arg, ld_shared_v4(stg + rr * 128 + (((lane & 7) ^ (rr & 7)) * 16)), e);
                            }
                            const int wrow = srow + r0;
                            const int wq = it.qi * p.tw + (wrow & (bw - 1)) + h * p.half_dq;
                            const int wp = it.pi * p.th + ((wrow >> p.bw_log2) & (bh - 1)) + h * p.half_dp;
                            const int wn = ni * p.tn + (wrow >> (p.bw_log2 + p.bh_log2));
                            if (col < p.Kout && wq < p.Q && wp < p.P && wn < p.N) {
                                const size_t po = ((static_cast<size_t>(wn) * (p.P >> 1) + (wp >> 1)) * (p.Q >> 1) + (wq >> 1)) * p.Kout + col;
                                *reinterpret_cast<float4*>(p.pool_out + po) = m;
                                if (p.pool_idx) *reinterpret_cast<uint32_t*>(p.pool_idx + po) = pool_code(m, arg);
                            }
                        }
                    }
                }
            } else if (kEpi == kEpiWarps && vec_ok) {
                // Coalesced path.  Each lane owns one row (pixel) of the accumulator, but a row's 32 columns
                // are 128 contiguous bytes in global memory, so the chunk is first transposed through a
                // 4 KB per-warp staging tile (XOR-swizzled 16-byte slots: conflict-free both ways) and then
                // written 4 rows x 128 bytes per instruction: lane l handles columns 4*(l&7).. of rows
                // (l>>3) + 4*i.  Bias, activation and the ReLU mask are applied on the way out.
                size_t roff[8];
                uint32_t vmask = 0;
                const size_t sp_off = static_cast<size_t>(it.sp) * p.split_stride;      // (0 unless the reduction is split)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int src = (lane >> 3) + 4 * i;
                    roff[i] = __shfl_sync(0xffffffffu, static_cast<unsigned long long>(pix_off + sp_off), src);
                    vmask |= (__shfl_sync(0xffffffffu, static_cast<int>(valid), src) ? 1u : 0u) << i;
                }
                const uint32_t stg = smem_u32(epi_stage + epi * 4096);
                const int cg = (lane & 7) * 4;
                for (int ch = ch0; ch < cpb; ch += kSub, ++cs_item) {
                    const int col = kt * p.BN + ch * 32 + cg;
                    // (the bias is fetched before the accumulator so that its latency hides behind the staging)
                    float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (p.bias && col < p.Kout) b = __ldg(reinterpret_cast<const float4*>(p.bias + col));
                    uint32_t v[32];
                    tmem_ld_32x32(t_row + ch * 32, v);
                    tmem_ld_wait();
                    if (!kPool && kEpi == kEpiWarps && p.split_acc) add_second_accumulator(t_row + t_second + ch * 32, v);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int slot = j ^ (lane & 7);
                        st_shared_v4(stg + lane * 128 + slot * 16, __uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                     __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    }
                    __syncwarp();
                    const unsigned live = __ballot_sync(0xffffffffu, col < p.Kout);   // lanes l, l^8, l^16 agree
                    if (col < p.Kout) {
                        // all eight staged rows first, so that their latencies overlap
                        float4 ov[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = (lane >> 3) + 4 * i;
                            ov[i] = ld_shared_v4(stg + rr * 128 + (((lane & 7) ^ (rr & 7)) * 16));
                        }
                        float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);
                        float4 mk[8];
                        if (kMask) {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                mk[i] = !((vmask >> i) & 1u) ? make_float4(0.f, 0.f, 0.f, 0.f)
                                        : p.mask_mode == 2 ? *reinterpret_cast<const float4*>(p.mask_src + roff[i] + col)   // (may be `out`)
                                                           : __ldg(reinterpret_cast<const float4*>(p.mask_src + roff[i] + col));
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float4 o = ov[i];
                            if ((vmask >> i) & 1u) {
                                o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
                                if (p.act == PCL_ACT_RELU) {
                                    o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f);
                                    o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f);
                                } else if (p.act == PCL_ACT_SIGMOID) {
                                    o.x = sigmoid_fast(o.x); o.y = sigmoid_fast(o.y);
                                    o.z = sigmoid_fast(o.z); o.w = sigmoid_fast(o.w);
                                }
                                if (kMask) {
                                    if (p.mask_mode == 0) {
                                        o.x = mk[i].x > 0.f ? o.x : 0.f; o.y = mk[i].y > 0.f ? o.y : 0.f;
                                        o.z = mk[i].z > 0.f ? o.z : 0.f; o.w = mk[i].w > 0.f ? o.w : 0.f;
                                    } else if (p.mask_mode == 2) {
                                        o.x = fmaf(-p.lr, o.x, mk[i].x); o.y = fmaf(-p.lr, o.y, mk[i].y);
                                        o.z = fmaf(-p.lr, o.z, mk[i].z); o.w = fmaf(-p.lr, o.w, mk[i].w);
                                    } else {
                                        o.x *= mk[i].x * (1.f - mk[i].x); o.y *= mk[i].y * (1.f - mk[i].y);
                                        o.z *= mk[i].z * (1.f - mk[i].z); o.w *= mk[i].w * (1.f - mk[i].w);
                                    }
                                }
                                *reinterpret_cast<float4*>(p.out + roff[i] + col) = o;
                                csum.x += o.x; csum.y += o.y; csum.z += o.z; csum.w += o.w;
                            }
                        }
                        if (p.colsum_cta) {
                            // (per-CTA sums: this lane's partial sums of the chunk are kept over the CTA's tiles, in
                            // the order of the tiles; the lane groups are added once, at the end)
                            if (cs_item == 0) { cacc0.x += csum.x; cacc0.y += csum.y; cacc0.z += csum.z; cacc0.w += csum.w; }
                            else if (cs_item == 1) { cacc1.x += csum.x; cacc1.y += csum.y; cacc1.z += csum.z; cacc1.w += csum.w; }
                            else if (cs_item == 2) { cacc2.x += csum.x; cacc2.y += csum.y; cacc2.z += csum.z; cacc2.w += csum.w; }
                            else { cacc3.x += csum.x; cacc3.y += csum.y; cacc3.z += csum.z; cacc3.w += csum.w; }
                        } else if (cs_row) {
                            // rows (lane>>3) + 4i were summed per lane; add the four lane groups in a fixed order
                            csum.x += __shfl_xor_sync(live, csum.x, 8);  csum.y += __shfl_xor_sync(live, csum.y, 8);
                            csum.z += __shfl_xor_sync(live, csum.z, 8);  csum.w += __shfl_xor_sync(live, csum.w, 8);
                            csum.x += __shfl_xor_sync(live, csum.x, 16); csum.y += __shfl_xor_sync(live, csum.y, 16);
                            csum.z += __shfl_xor_sync(live, csum.z, 16); csum.w += __shfl_xor_sync(live, csum.w, 16);
                            if (lane < 8) *reinterpret_cast<float4*>(cs_row + col) = csum;
                        }
                        if (kPool) {
                            // Fused 2x2 max pooling.  The warp's 32 rows are 32 consecutive pixels of the box
                            // (bit 0 of the row = parity of q, bit log2(bw) = parity of p; the box starts at even
                            // coordinates), so they hold 8 whole windows; lane l takes windows (l >> 3) and
                            // (l >> 3) + 4 of its 4 columns.  max commutes with adding the bias and with the
                            // (monotone) activation, so the maximum of the raw accumulators is finished like `o`.
                            const int lb = p.bw_log2;
#pragma unroll
                            for (int half = 0; half < 2; ++half) {
                                const int wdx = (lane >> 3) + 4 * half;
                                const int r0 = ((wdx & ((1 << (lb - 1)) - 1)) << 1) | ((wdx >> (lb - 1)) << (lb + 1));
                                // (the staged values are raw accumulators here: each is finished like `o` before it is compared)
                                float4 m = finish4(ld_shared_v4(stg + r0 * 128 + (((lane & 7) ^ (r0 & 7)) * 16)), b, p.act);
                                uint32_t arg = 0;
#pragma unroll
                                for (int e = 1; e < 4; ++e) {
                                    const int rr = r0 | (e & 1) | ((e >> 1) << lb);
                                    pool_take(m, arg, finish4(ld_shared_v4(stg + rr * 128 + (((lane & 7) ^ (rr & 7)) * 16)), b, p.act), e);
                                }
                                const int wrow = quarter * 32 + r0;       // the window's first pixel inside the box
                                const int wq = it.qi * p.tw + (wrow & (bw - 1)) + h * p.half_dq;
                                const int wp = it.pi * p.th + ((wrow >> p.bw_log2) & (bh - 1)) + h * p.half_dp;
                                const int wn = ni * p.tn + (wrow >> (p.bw_log2 + p.bh_log2));
                                if (wq < p.Q && wp < p.P && wn < p.N) {
                                    const size_t po = ((static_cast<size_t>(wn) * (p.P >> 1) + (wp >> 1)) * (p.Q >> 1) + (wq >> 1)) * p.Kout + col;
                                    *reinterpret_cast<float4*>(p.pool_out + po) = m;
                                    if (p.pool_idx) *reinterpret_cast<uint32_t*>(p.pool_idx + po) = pool_code(m, arg);
                                }
                            }
                        }
                    }
                    __syncwarp();
                }
            } else if (kEpi == kEpiWarps) {
                for (int ch = ch0; ch < cpb; ch += kSub) {
                    uint32_t v[32];
                    tmem_ld_32x32(t_row + ch * 32, v);
                    tmem_ld_wait();
                    if (!kPool && kEpi == kEpiWarps && p.split_acc) add_second_accumulator(t_row + t_second + ch * 32, v);
                    const int col0 = kt * p.BN + ch * 32;
                    if (valid && col0 < p.Kout) {
                        float* dst = p.out + static_cast<size_t>(it.sp) * p.split_stride + pix_off + col0;
                        const float* msk = kMask ? p.mask_src + pix_off + col0 : nullptr;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (col0 + j < p.Kout) {
                                float o = __uint_as_float(v[j]);
                                if (p.bias) o += __ldg(p.bias + col0 + j);
                                if (p.act == PCL_ACT_RELU) o = fmaxf(o, 0.f);
                                else if (p.act == PCL_ACT_SIGMOID) o = sigmoid_fast(o);
                                if (msk) {
                                    const float m = p.mask_mode == 2 ? msk[j] : __ldg(msk + j);
                                    o = p.mask_mode == 0 ? (m > 0.f ? o : 0.f) : (p.mask_mode == 2 ? fmaf(-p.lr, o, m) : o * (m * (1.f - m)));
                                }
                                dst[j] = o;
                            }
                        }
                    }
                }
            }
            }   // halves
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (kPair && pair_rank != 0) mbar_arrive_cluster(map_to_cta(&tmem_empty_bar[acc], 0));
                else mbar_arrive(&tmem_empty_bar[acc]);
            }
        }
        if (!kMask && p.tma_store && lane == 0) bulk_wait_group0();     // every store of this warp has completed
        if (p.colsum_cta && p.colsum_rows) {
            // one row per (CTA, box, lane quarter): the four lane groups of each chunk are added in a fixed order
            int item = 0;
            for (int h = 0; h < p.MT; ++h)
                for (int ch = (sub - h * cpb) & (kSub - 1); ch < cpb; ch += kSub, ++item) {
                    float4 c = item == 0 ? cacc0 : (item == 1 ? cacc1 : (item == 2 ? cacc2 : cacc3));
                    c.x += __shfl_xor_sync(0xffffffffu, c.x, 8);  c.y += __shfl_xor_sync(0xffffffffu, c.y, 8);
                    c.z += __shfl_xor_sync(0xffffffffu, c.z, 8);  c.w += __shfl_xor_sync(0xffffffffu, c.w, 8);
                    c.x += __shfl_xor_sync(0xffffffffu, c.x, 16); c.y += __shfl_xor_sync(0xffffffffu, c.y, 16);
                    c.z += __shfl_xor_sync(0xffffffffu, c.z, 16); c.w += __shfl_xor_sync(0xffffffffu, c.w, 16);
                    const int col = ch * 32 + (lane & 7) * 4;      // (tiles_k == 1: every tile has these columns)
                    if (lane < 8 && col < p.Kout)
                        *reinterpret_cast<float4*>(p.colsum_rows + ((static_cast<size_t>(blockIdx.x) * p.MT + h) * 4 + quarter) * p.Kout + col) = c;
                }
        }
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync_all();     // neither CTA leaves while the pair's MMAs or arrivals may touch it
    if (warp == 1) {
        tc_fence_after();
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, p.tmem_cols);
        else tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// Pick the 128-pixel box bw x bh x bn (powers of two) that wastes the least
// work on ragged edges; ties go to the widest box.
// pool: the box must hold whole 2x2 windows inside each 32-pixel quarter (2 <= bw <= 16, bh >= 2).
// stride_w / stride_h: a TMA box spans bw * stride_w x bh * stride_h input pixels, at most 256 each.
void choose_box(int P, int Q, int N, bool pool, int* bw_log2, int* bh_log2, int stride_w = 1, int stride_h = 1) {
    double best = 1e300;
    int best_w = pool ? 1 : 0, best_h = pool ? 1 : 0;
    for (int lw = pool ? 4 : 7; lw >= (pool ? 1 : 0); --lw)
        for (int lh = 7 - lw; lh >= (pool ? 1 : 0); --lh) {
            const long bw = 1L << lw, bh = 1L << lh, bn = 128 / (bw * bh);
            if (bw * stride_w > 256 || bh * stride_h > 256) continue;
            const double covered = double((Q + bw - 1) / bw * bw) * double((P + bh - 1) / bh * bh) *
                                   double((N + bn - 1) / bn * bn);
            if (covered < best) { best = covered; best_w = lw; best_h = lh; }
        }
    *bw_log2 = best_w;
    *bh_log2 = best_h;
}

int choose_bn(int Kout, long m_tiles, int sm_count) {
    if (tune_is_set(TUNE_BN)) {          // tuning hook: a multiple of 32 in [32, 256]
        const int bn = tune(TUNE_BN, 0);
        if (bn >= 32 && bn <= 256 && bn % 32 == 0) return bn;
    }
    // Score = (fraction of SM-slots the tiles fill, counting whole waves) x (tensor efficiency of the width):
    // an MMA costs max(N/2, ~52) cycles, so N < 128 wastes the pipe, and wider tiles re-read A less often.
    const int k32 = (Kout + 31) / 32 * 32;
    int best = 32;
    double best_score = -1.0;
    for (int bn = 256; bn >= 32; bn -= 32) {
        if (bn > k32 && bn != 32) continue;
        const long n_tiles = (Kout + bn - 1) / bn;
        if ((n_tiles - 1) * bn >= Kout) continue;
        // balance the last tile: Kout = 1000 -> 4 x 256 rather than 3 x 256 + 232
        const int bal = int(((Kout + n_tiles - 1) / n_tiles + 31) / 32 * 32);
        if (bal != bn && bal < bn) continue;       // the balanced width is tried on its own
        const long tiles = m_tiles * n_tiles;
        const long waves = (tiles + sm_count - 1) / sm_count;
        const double fill = double(tiles) / double(waves * sm_count);
        const double useful = double(Kout) / double(n_tiles * bn);           // ragged last columns
        const double eff = (bn >= 128 ? 0.88 + 0.12 * (bn - 128) / 128.0 : 0.88 * bn / 128.0);
        const double score = fill * useful * eff;
        if (score > best_score + 1e-9) { best_score = score; best = bn; }
    }
    return best;
}

}  // namespace

bool tc_fprop_can_pool(const TcFpropArgs& a) {
    return a.P % 2 == 0 && a.Q % 2 == 0 && a.P >= 2 && a.Q >= 2 && a.Kout % 4 == 0 && a.mask_src == nullptr;
}

bool tc_fprop_eligible(const TcFpropArgs& a) {
    if (a.wt_mn_major && a.Kout % kBlockC != 0) return false;
    if (a.Cin % 4 != 0) return false;                       // TMA strides are multiples of 16 bytes
    if ((reinterpret_cast<uintptr_t>(a.in) | reinterpret_cast<uintptr_t>(a.wt)) & 15) return false;
    if (a.R * a.S > 65535) return false;
    if (a.stride_h < 1 || a.stride_w < 1 || a.stride_h > 8 || a.stride_w > 8 || a.dil_w < 1) return false;
    if ((a.out_stride_w | a.out_stride_h | a.out_stride_n) != 0 && (a.pool_out || a.split_ws)) return false;
    return true;
}

namespace {

// One way of tiling a layer: plain (a box of 128 pixels, one TMA box per tap) or halo (MT boxes of 8 x 16
// pixels cut from one haloed patch per channel block).

struct TileCfg {
    bool ok = false;
    int halo = 0, MT = 1, bw_log2 = 0, bh_log2 = 0, tw = 0, th = 0, tn = 0, half_dq = 0, half_dp = 0;
    int tiles_q = 0, tiles_p = 0, tiles_n = 0, tiles_k = 0, BN = 0;
    int PW = 0, patch_bytes = 0, a_buf_bytes = 0, NA = 0, half_off_bytes = 0, stages = 0, KS = 1;
    int issuers = 1;    // MMA-issuing threads
    int grp = 0;        // one copy per operand and slot (KS channel blocks of one tap)
    int pair = 0;       // CTA pairs: two image-group tiles share one 256-wide weight tile (see the kernel)
};

// bn_force / pair_force (-1 = the builder's own rule): the candidates the blocking search enumerates
TileCfg plain_cfg(const TcFpropArgs& a, int cblocks, int sm_count, int bn_force = -1, int pair_force = -1) {
    TileCfg c;
    choose_box(a.P, a.Q, a.N, a.pool_out != nullptr, &c.bw_log2, &c.bh_log2, a.stride_w, a.stride_h);
    c.tw = 1 << c.bw_log2; c.th = 1 << c.bh_log2; c.tn = kTileM / (c.tw * c.th);
    c.tiles_q = (a.Q + c.tw - 1) / c.tw; c.tiles_p = (a.P + c.th - 1) / c.th; c.tiles_n = (a.N + c.tn - 1) / c.tn;
    const long m_tiles = long(c.tiles_q) * c.tiles_p * c.tiles_n;
    c.BN = bn_force > 0 ? bn_force : choose_bn(a.Kout, m_tiles, sm_count);
    c.tiles_k = (a.Kout + c.BN - 1) / c.BN;
    // narrow tiles: several k-steps per slot (see the kernel), as long as 4 slots still fit
    // pairs pay where operand traffic or the issue rate of wide MMAs bounds the tile; narrow tiles are bound by
    // the issuing thread and run as single CTAs with two issuers instead
    const bool pair_ok = c.BN >= 64 && c.BN % 16 == 0 && c.tiles_n >= 2 && sm_count >= 2 &&
                         (!a.wt_mn_major || c.BN % 64 == 0);    // MN-major weights are fetched in whole 32-map groups per CTA
    c.pair = pair_force >= 0 ? (pair_force && pair_ok) : (tune(TUNE_PAIR, 1) && c.BN >= 128 && pair_ok);
    const int step_bytes = kABytes + (c.pair ? c.BN * 64 : c.BN * 128);
    c.KS = tune(TUNE_KS, 2);
    const int kiters = a.R * a.S * cblocks;
    if (c.KS > kiters) c.KS = kiters;
    while (c.KS > 1 && (kSmemBudget - kEpiStageBytes) / (c.KS * step_bytes) < 3) --c.KS;
    c.stages = (kSmemBudget - kEpiStageBytes) / (c.KS * step_bytes);
    c.grp = tune(TUNE_GRP, 1) && c.KS > 1 && a.Cin % kBlockC == 0 && cblocks % c.KS == 0 && a.in_inner == 0;
    if (c.stages > kMaxStages) c.stages = kMaxStages;
    c.ok = c.stages >= 2;
    return c;
}

// layout: 0 = one box (8 x 16), 1 = two boxes side by side (16 x 16), 2 = two boxes stacked (8 x 32)
TileCfg halo_cfg(const TcFpropArgs& a, int cblocks, int sm_count, int layout, int bn_force = -1, int pair_force = -1) {
    TileCfg c;
    c.halo = 1; c.MT = layout == 0 ? 1 : 2;
    c.bw_log2 = 3; c.bh_log2 = 4;
    c.tw = layout == 1 ? 16 : 8; c.th = layout == 2 ? 32 : 16; c.tn = 1;
    c.half_dq = layout == 1 ? 8 : 0; c.half_dp = layout == 2 ? 16 : 0;
    c.PW = c.tw + a.S - 1;
    const int PH = c.th + a.R - 1;
    if (a.R * a.S <= 1 || c.PW > 256 || PH > 256) return c;
    if (a.stride_h != 1 || a.stride_w != 1 || a.dil_w != 1) return c;      // taps as shifted views need unit steps
    c.patch_bytes = c.PW * PH * 128;
    c.a_buf_bytes = (c.patch_bytes + 1023) / 1024 * 1024;
    c.half_off_bytes = layout == 1 ? 8 * 128 : (layout == 2 ? 16 * c.PW * 128 : 0);
    c.tiles_q = (a.Q + c.tw - 1) / c.tw; c.tiles_p = (a.P + c.th - 1) / c.th; c.tiles_n = a.N;
    const long m_tiles = long(c.tiles_q) * c.tiles_p * c.tiles_n;
    c.BN = bn_force > 0 ? bn_force : choose_bn(a.Kout, m_tiles, sm_count);
    if (2 * c.MT * c.BN > 512) return c;          // two accumulator sets must fit the 512 TMEM columns
    c.tiles_k = (a.Kout + c.BN - 1) / c.BN;
    // Pairs of images: the two CTAs of a cluster take the same tile of two consecutive images against the same weight
    // tile, of which each loads half the rows (the conditions are the plain tiling's: whole 16-column MMA halves,
    // MN-major weights in whole 32-map groups per CTA).  Halving the weight bytes per CTA doubles the depth of the
    // weight ring, which is what a narrow layer's tiles wait for.
    const bool pair_ok = c.BN >= 64 && c.BN % 16 == 0 && c.tiles_n >= 2 && sm_count >= 2 && (!a.wt_mn_major || c.BN % 64 == 0);
    c.pair = (pair_force >= 0 ? pair_force != 0 : tune(TUNE_PAIR_HALO, 0) != 0) && pair_ok;
    const int b_bytes = c.pair ? c.BN * 64 : c.BN * 128;
    const int room = kSmemBudget - kEpiStageBytes;
    c.NA = 2;
    c.KS = tune(TUNE_KS_HALO, (c.BN <= 64 || (c.pair && c.BN <= 128)) ? 3 : (c.BN <= 128 ? 2 : 1));
    if (c.KS > a.R * a.S) c.KS = a.R * a.S;
    while (c.KS > 1 && (room - c.NA * c.a_buf_bytes) / (c.KS * b_bytes) < 3) --c.KS;
    c.grp = tune(TUNE_GRP, 1) && c.KS > 1 && !a.wt_mn_major;      // (MN-major weights: one copy per tap)
    const int slot = c.KS * b_bytes;
    c.stages = (room - c.NA * c.a_buf_bytes) / slot;
    if (c.stages >= 9 && (room - 3 * c.a_buf_bytes) / slot >= 6) {
        c.NA = 3;
        c.stages = (room - 3 * c.a_buf_bytes) / slot;
    }
    if (c.stages > kMaxStages) c.stages = kMaxStages;
    if (c.stages < 3) return c;
    c.ok = true;
    return c;
}

// ---- Blocking search (Sec. 2.2 / 2.3 re-posed for this memory hierarchy) ------------------------------------------
// The paper chooses its cache and register blocks by minimising the bytes moved per flop under the capacity of the
// cache, with a brute-force search over the block sizes.  Here the scarce rates are the tensor pipe, the fill rate
// of shared memory out of L2, the issuing warp and the epilogue warps, under 227 KB of shared memory and 512
// TMEM columns; a candidate's cost is the slowest of those four per tile, times the tiles a CTA takes.  Constants
// are measurements on B200 (microbenchmarks and ncu captures of these kernels).
struct TileCost { double mma, fill, issue, epilogue, tile, total; };
constexpr double kMmaFloorClk = 52.0;        // a K = 8 MMA of N columns takes max(N / 2, 52) cycles
constexpr double kFillSingle = 60.0;         // bytes per clock and SM into shared memory, single CTAs of this kernel
constexpr double kFillPair = 57.0;           //   ... CTA pairs (which need a third fewer bytes per MMA)
constexpr double kHaloMmaFactor = 1.5;       // haloed tiles take this much longer than their MMAs (a fit: the pipe itself runs row-shifted views at full rate)
constexpr double kHaloPairMmaFactor = 1.3;   //   ... as CTA pairs (half the weight bytes per CTA, a weight ring twice as deep)
constexpr double kHaloOneBoxFactor = 1.3;    //   ... and slower still when a tile is one box (no second box to share a weight tile with)
constexpr double kIssueMmaClk = 45.0;        // the issuing thread's cost per MMA
constexpr double kIssueSlotClk = 160.0;      //   ... per pipeline slot (one barrier round trip and one commit)
constexpr double kEpilogueChunkClk = 1600.0; // an epilogue warp's cost per 32 x 32 chunk
constexpr double kTileFixedClk = 300.0, kLaunchFixedClk = 4000.0;

TileCost predict_cost(const TcFpropArgs& a, const TileCfg& c, int cblocks, int sm_count) {
    TileCost t{};
    const double ksteps = double(a.R) * a.S * cblocks;
    const double b_bytes = c.pair ? c.BN * 64.0 : c.BN * 128.0;
    const double mma_clk = c.BN / 2.0 > kMmaFloorClk ? c.BN / 2.0 : kMmaFloorClk;
    t.mma = c.MT * ksteps * 4.0 * mma_clk * (c.halo ? (c.pair ? kHaloPairMmaFactor : kHaloMmaFactor) * (c.MT == 1 ? kHaloOneBoxFactor : 1.0) : 1.0);
    const double bytes = c.halo ? cblocks * (double(c.patch_bytes) + double(a.R) * a.S * b_bytes) : ksteps * (kABytes + b_bytes);
    t.fill = bytes / (c.pair ? kFillPair : kFillSingle);
    const double slots = c.halo ? cblocks * double((a.R * a.S + c.KS - 1) / c.KS) : (ksteps + c.KS - 1) / c.KS;
    const int issuers = (!c.pair && slots >= 8) ? 2 : 1;
    t.issue = (c.MT * ksteps * 4.0 * kIssueMmaClk + slots * kIssueSlotClk) / issuers;
    const double chunks = c.MT * (c.BN / 32.0) * 4.0;
    t.epilogue = double(long((chunks + kEpiWarps - 1) / kEpiWarps)) * kEpilogueChunkClk * (a.pool_out ? 1.3 : 1.0);
    t.tile = t.mma;
    if (t.fill > t.tile) t.tile = t.fill;
    if (t.issue > t.tile) t.tile = t.issue;
    if (t.epilogue > t.tile) t.tile = t.epilogue;
    t.tile += kTileFixedClk;
    const double m_tiles = double(c.tiles_q) * c.tiles_p * (c.pair ? (c.tiles_n + 1) / 2 : c.tiles_n);
    const double work_items = m_tiles * c.tiles_k;                       // CTA tiles (a pair's two tiles count once)
    const double slots_sm = c.pair ? sm_count / 2 : sm_count;
    const double per_cta = double(long((work_items + slots_sm - 1) / slots_sm));
    t.total = per_cta * t.tile + kLaunchFixedClk;
    return t;
}

// Enumerates the candidate tilings of a launch -- plain tiling x tile width x single CTAs or pairs, the three haloed
// layouts x tile width -- and returns the one the cost model predicts fastest.
TileCfg search_cfg(const TcFpropArgs& a, int sm_count, TileCost* best_cost = nullptr) {
    const int cblocks = (a.Cin + kBlockC - 1) / kBlockC;
    TileCfg best;
    double best_total = 1e300;
    const int k32 = (a.Kout + 31) / 32 * 32;
    // (one tile width beyond the output's: a layer of 96 maps also tries 128-wide tiles, whose last 32 columns multiply
    // zero fill and are not stored, because only multiples of 64 can run as CTA pairs)
    const int k64 = (a.Kout + 63) / 64 * 64;
    for (int bn = 32; bn <= 256; bn += 32) {
        if (bn > k32 && bn != k64) break;
        if (a.wt_mn_major && (a.Kout % 32 != 0)) break;
        const int n_tiles = (a.Kout + bn - 1) / bn;
        if ((n_tiles - 1) * bn >= a.Kout) continue;
        const int halo_pairs = tune(TUNE_PAIR_HALO, 1) ? 3 : 0;      // (PAIR_HALO = 0 takes the paired haloed candidates out)
        for (int variant = 0; variant < 5 + halo_pairs; ++variant) {
            const TileCfg c = variant < 2 ? plain_cfg(a, cblocks, sm_count, bn, variant)
                              : variant < 5 ? halo_cfg(a, cblocks, sm_count, variant - 2, bn, 0)
                                            : halo_cfg(a, cblocks, sm_count, variant - 5, bn, 1);
            if (!c.ok || ((variant == 1 || variant >= 5) && !c.pair)) continue;
            if (c.halo && a.pool_out && (c.bw_log2 < 1 || c.bh_log2 < 1)) continue;
            const TileCost t = predict_cost(a, c, cblocks, sm_count);
            // (a haloed candidate must beat the plain ones by a tenth: its prediction is the less certain one)
            // (and between a haloed candidate and its paired form, which the model prices alike, the pair wins: it
            // fetches half the weight bytes per CTA)
            const double score = t.total * (c.halo ? (c.pair ? 1.099 : 1.1) : 1.0);
            if (score < best_total) { best_total = score; best = c; if (best_cost) *best_cost = t; }
        }
    }
    return best;
}

// The tiling a launch will use (also needed to size the fused column-sum rows).
TileCfg select_cfg(const TcFpropArgs& a, int sm_count) {
    const int cblocks = (a.Cin + kBlockC - 1) / kBlockC;
    // Convolutions (more than one tap) take the candidate the cost model predicts fastest; measured against every
    // candidate (python -m paper_1602_06709_b200.blocking_search) it is within a few percent of the measured best on
    // every VGG-A and OverFeat-FAST layer at minibatch 256.  1 x 1 layers (the FC GEMMs) keep the rules below, which also decide their reduction splits.
    // SELECT = 0 switches the model off, 1 applies it to every launch; a pinned knob always wins.
    // (the few-channel path reads overlapping windows, whose fill cost the model does not describe: rules too)
    const int sel = tune(TUNE_SELECT, (a.R * a.S > 1 && a.in_stride_w == 0) ? 1 : 0);
    if (sel == 1 && tune(TUNE_TILING, -1) < 0 && !tune_is_set(TUNE_BN) && !tune_is_set(TUNE_PAIR) && !tune_is_set(TUNE_KS) &&
        !tune_is_set(TUNE_KS_HALO) && !tune_is_set(TUNE_GRP) && tune(TUNE_PAIR_HALO, 0) == 0) {
        const TileCfg m = search_cfg(a, sm_count);
        if (m.ok) return m;
    }
    TileCfg cfg = plain_cfg(a, cblocks, sm_count);
    if (!cfg.ok) return cfg;
    // Test hook: the TILING knob pins the tiling (when that tiling is possible).
    const int pin = tune(TUNE_TILING, -1);       // unset: the rule below; 0: plain; 1-3: haloed layout 0-2
    const int pinned = pin < 0 || pin > 3 ? -2 : pin - 1;
    for (int layout = 0; layout < 3; ++layout) {
        const TileCfg h = halo_cfg(a, cblocks, sm_count, layout);
        if (!h.ok) continue;
        if (pinned == layout) { cfg = h; break; }
        // Measured on B200: the haloed tiling only pays where the plain one is starved by operand traffic,
        // i.e. narrow layers (BN <= 128) tiled without ragged edges by two boxes that share every weight tile;
        // wide layers already run at the power-limited tensor rate with the plain tiling.
        if (pinned == -2 && layout > 0 && h.BN <= 128 && a.Q % h.tw == 0 && a.P % h.th == 0) { cfg = h; break; }
    }
    return cfg;
}

}  // namespace

// Rows of column sums the launch for `a` writes (rows 0 .. n-1 of its colsum_rows buffer): per CTA where every tile
// has the same columns, else per tile.
long tc_fprop_colsum_rows_written(const TcFpropArgs& a, bool* all_written) {
    const int sm = device_sm_count();
    if (all_written) *all_written = false;
    if (a.Kout % 4 != 0) return 0;
    const TileCfg c = select_cfg(a, sm);
    if (!c.ok) return 0;
    if (c.tiles_k == 1) return long(sm) * c.MT * 4;       // (a grid smaller than the device leaves rows untouched)
    // per tile: every row is written, unless a pair's last half is an image group that does not exist
    if (all_written) *all_written = !(c.pair && (c.tiles_n & 1));
    return long(c.tiles_q) * c.tiles_p * c.tiles_n * c.MT * 4;
}

long tc_fprop_colsum_rows(const TcFpropArgs& a) {
    const int sm = device_sm_count();
    if (a.Kout % 4 != 0) return 0;
    // rows are independent of BN, but the haloed / plain choice depends on it: take the larger of all tilings
    long rows = 0;
    const int cblocks = (a.Cin + kBlockC - 1) / kBlockC;
    const TileCfg pc = plain_cfg(a, cblocks, sm);
    if (pc.ok) rows = long(pc.tiles_q) * pc.tiles_p * pc.tiles_n * 4;
    for (int layout = 0; layout < 3; ++layout) {
        const TileCfg h = halo_cfg(a, cblocks, sm, layout);
        const long r = h.ok ? long(h.tiles_q) * h.tiles_p * h.tiles_n * h.MT * 4 : 0;
        if (r > rows) rows = r;
    }
    return rows;
}

namespace {
// Reduction splits for a launch with few tiles and a long reduction (plain tiling, no fused mask / sums / pooling):
// as many as fill the SMs, each an equal whole number of pipeline slots (at least two).
int choose_ksplit(const TcFpropArgs& a, const TileCfg& cfg, int cblocks, int sm_count) {
    if (cfg.halo || a.mask_src || a.colsum_rows || a.pool_out || !a.out || a.Kout % 4 != 0) return 1;
    const int hook = tune(TUNE_KSPLIT, 0);              // test hook: 1 = never, n = n splits where they divide
    if (hook == 1) return 1;
    const long tiles = long(cfg.tiles_q) * cfg.tiles_p * cfg.tiles_n * cfg.tiles_k;        // CTAs (a pair is two)
    const int kiters = a.R * a.S * cblocks;
    if (kiters % cfg.KS != 0) return 1;
    const int slots = kiters / cfg.KS;
    long want = hook > 1 ? hook : sm_count / tiles;
    if (want > 32) want = 32;
    // measured (B200, minibatch 256): the second pass costs ~5 us, which splitting repays from ~32 slots on
    // (C = 2048) when each split keeps at least 8
    if (hook <= 1 && (tiles * 2 > sm_count || slots < 32)) return 1;
    const int min_slots = hook > 1 ? 2 : 8;
    for (int k = int(want); k >= 2; --k)
        if (slots % k == 0 && slots / k >= min_slots) return k;
    return 1;
}
}  // namespace

int tc_fprop_describe(const TcFpropArgs& a, char* buf, size_t n) {
    if (!tc_fprop_eligible(a)) return PCL_ERR_UNSUPPORTED_SHAPE;
    const int sm = device_sm_count();
    const int cblocks = (a.Cin + kBlockC - 1) / kBlockC;
    const TileCfg c = select_cfg(a, sm);
    if (!c.ok) return PCL_ERR_UNSUPPORTED_SHAPE;
    const TileCost t = predict_cost(a, c, cblocks, sm);
    TileCost mt{};
    const TileCfg m = search_cfg(a, sm, &mt);
    const char* names[4] = {"plain", "halo0", "halo1", "halo2"};
    auto name = [&](const TileCfg& x) { return names[!x.halo ? 0 : (x.MT == 1 ? 1 : (x.half_dq ? 2 : 3))]; };
    snprintf(buf, n,
             "tiling=%s BN=%d pair=%d KS=%d stages=%d box=%dx%dx%d predicted_clk=%.0f (mma %.0f fill %.0f issue %.0f epilogue %.0f per "
             "tile) | model_choice: tiling=%s BN=%d pair=%d predicted_clk=%.0f",
             name(c), c.BN, c.pair, c.KS, c.stages, c.tw, c.th, c.tn, t.total, t.mma, t.fill, t.issue, t.epilogue, name(m), m.BN,
             m.pair, mt.total);
    return PCL_OK;
}

size_t tc_fprop_split_ws_bytes(const TcFpropArgs& a) {
    const int sm = device_sm_count();
    if (!tc_fprop_eligible(a)) return 0;
    const TileCfg cfg = select_cfg(a, sm);
    if (!cfg.ok) return 0;
    TcFpropArgs b = a;
    if (!b.out) b.out = reinterpret_cast<float*>(16);       // (sizing query: only "an output exists" matters)
    const int k = choose_ksplit(b, cfg, (a.Cin + kBlockC - 1) / kBlockC, sm);
    return k > 1 ? size_t(k) * a.N * a.P * a.Q * a.Kout * 4 : 0;
}

namespace {
// Everything a launch needs that follows from its arguments alone (tiling, kernel parameters, tensor maps, grid):
// built once per distinct argument set and kept (see launch_tc_fprop).
struct FpropPlan {
    FpropParams p;
    CUtensorMap tmA, tmB, tmOut;
    bool pair = false, wide_epi = false;
    size_t smem = 0;
    long total = 0;          // CTA tiles (pair: pair tiles)
    int sm_count = 0, grid = 0;
    double flops = 0.0;
};
int build_fprop_plan(const TcFpropArgs& a, FpropPlan* plan);
int run_fprop_plan(const FpropPlan& plan, const TcFpropArgs& a, cudaStream_t st);

// Plan cache.  The key is every field of the arguments (pointers included: they are in the tensor maps), the device and
// the generation of the tuning knobs; a step driver that calls with the same buffers every step pays for tiling
// selection and three cuTensorMapEncodeTiled calls once per layer and pass instead of once per call.
void key_put(std::string& k, const void* v, size_t n) { k.append(static_cast<const char*>(v), n); }
template <class T> void key_put(std::string& k, const T& v) { key_put(k, &v, sizeof(T)); }
std::string fprop_plan_key(const TcFpropArgs& a, int device) {
    std::string k;
    k.reserve(320);
    key_put(k, a.in); key_put(k, a.wt); key_put(k, a.bias); key_put(k, a.mask_src); key_put(k, a.out);
    const int ints[] = {a.N, a.H, a.W, a.Cin, a.Kout, a.R, a.S, a.pad_h, a.pad_w, a.P, a.Q, a.act, a.mask_mode, a.k_live, a.in_inner,
                        a.wt_mn_major, a.flip_taps, a.stride_h, a.stride_w, a.dil_w, device};
    key_put(k, ints, sizeof(ints));
    const long longs[] = {a.in_stride_w, a.in_stride_h, a.in_stride_n, a.out_stride_w, a.out_stride_h, a.out_stride_n};
    key_put(k, longs, sizeof(longs));
    key_put(k, a.lr); key_put(k, a.colsum_rows); key_put(k, a.pool_out); key_put(k, a.pool_idx); key_put(k, a.split_ws);
    key_put(k, a.split_ws_bytes);
    const unsigned long long gen = tune_generation();
    key_put(k, gen);
    return k;
}
std::mutex g_plan_mu;
std::unordered_map<std::string, FpropPlan> g_plans;
std::atomic<unsigned long long> g_plan_hits{0}, g_plan_misses{0};
constexpr size_t kMaxPlans = 512;       // (a network has a few dozen distinct launches; beyond this the cache starts over)
}  // namespace

void plan_cache_count(bool hit) { if (hit) ++g_plan_hits; else ++g_plan_misses; }

void plan_cache_stats(unsigned long long* hits, unsigned long long* misses) {
    if (hits) *hits = g_plan_hits.load();
    if (misses) *misses = g_plan_misses.load();
}

int launch_tc_fprop(const TcFpropArgs& a, cudaStream_t st) {
    if (!tune(TUNE_PLAN_CACHE, 1)) {
        FpropPlan plan;
        const int rc = build_fprop_plan(a, &plan);
        return rc != PCL_OK ? rc : run_fprop_plan(plan, a, st);
    }
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return PCL_ERR_CUDA;
    const std::string key = fprop_plan_key(a, device);
    FpropPlan plan;
    bool hit = false;
    {
        std::lock_guard<std::mutex> lock(g_plan_mu);
        auto it = g_plans.find(key);
        if (it != g_plans.end()) { plan = it->second; hit = true; }
    }
    plan_cache_count(hit);
    if (!hit) {
        const int rc = build_fprop_plan(a, &plan);
        if (rc != PCL_OK) return rc;
        std::lock_guard<std::mutex> lock(g_plan_mu);
        if (g_plans.size() >= kMaxPlans) g_plans.clear();
        g_plans.emplace(key, plan);
    }
    return run_fprop_plan(plan, a, st);
}

namespace {
int build_fprop_plan(const TcFpropArgs& a, FpropPlan* plan) {
    if (!tc_fprop_eligible(a)) return PCL_ERR_UNSUPPORTED_SHAPE;
    static PerDeviceOnce attr_once;       // (the attribute applies to the current device only)
    const int setup_rc = attr_once.run([]() -> int {
        const void* kernels[8] = {
            (const void*)tc_fprop_kernel<false, false, false>, (const void*)tc_fprop_kernel<false, true, false>,
            (const void*)tc_fprop_kernel<false, false, true>,  (const void*)tc_fprop_kernel<true, false, false>,
            (const void*)tc_fprop_kernel<true, true, false>,   (const void*)tc_fprop_kernel<true, false, true>,
            (const void*)tc_fprop_kernel<false, false, false, kEpiWarpsWide>,
            (const void*)tc_fprop_kernel<false, true, false, kEpiWarpsWide>};
        for (const void* k : kernels)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024) != cudaSuccess)
                return PCL_ERR_CUDA;
        return PCL_OK;
    });
    if (setup_rc != PCL_OK) return setup_rc;
    const int g_sm_count = device_sm_count();
    FpropParams p{};
    p.cblocks = (a.Cin + kBlockC - 1) / kBlockC;
    const TileCfg cfg = select_cfg(a, g_sm_count);
    if (!cfg.ok) return PCL_ERR_UNSUPPORTED_SHAPE;
    p.halo = cfg.halo; p.MT = cfg.MT; p.bw_log2 = cfg.bw_log2; p.bh_log2 = cfg.bh_log2;
    p.tw = cfg.tw; p.th = cfg.th; p.tn = cfg.tn; p.half_dq = cfg.half_dq; p.half_dp = cfg.half_dp;
    p.tiles_q = cfg.tiles_q; p.tiles_p = cfg.tiles_p; p.tiles_k = cfg.tiles_k;
    p.tiles_n = cfg.pair ? (cfg.tiles_n + 1) / 2 : cfg.tiles_n;      // pair mode iterates over pairs of image groups
    p.BN = cfg.BN; p.PW = cfg.PW; p.patch_bytes = cfg.patch_bytes; p.a_buf_bytes = cfg.a_buf_bytes; p.NA = cfg.NA;
    p.half_off_bytes = cfg.half_off_bytes; p.stages = cfg.stages; p.KS = cfg.KS; p.grp = cfg.grp;
    p.bmn = a.wt_mn_major ? 1 : 0; p.flip = a.flip_taps ? 1 : 0;
    // Two issuing threads only for single-CTA tiles: pair MMAs (cta_group::2) issued from two warps at once
    // ended in launch failures on B200, so a pair always has one issuer.
    // They pay where a tile has many slots; the hand-over between the threads costs more than it hides on
    // tiles of a few k-steps (the few-channel first layer: 3).
    const int slots_per_tile = cfg.halo ? p.cblocks * ((a.R * a.S + cfg.KS - 1) / cfg.KS)
                                        : (a.R * a.S * p.cblocks + cfg.KS - 1) / cfg.KS;
    p.issuers = (!cfg.pair && slots_per_tile >= 8 && tune(TUNE_ISSUERS, 2) >= 2) ? 2 : 1;
    const int bw = 1 << p.bw_log2, bh = 1 << p.bh_log2, bn = kTileM / (bw * bh);
    const long m_tiles = long(p.tiles_q) * p.tiles_p * p.tiles_n;
    if (m_tiles * p.tiles_k > 0x7fffffffL) return PCL_ERR_UNSUPPORTED_SHAPE;
    p.R = a.R; p.S = a.S; p.pad_h = a.pad_h; p.pad_w = a.pad_w;
    p.stride_h = a.stride_h; p.stride_w = a.stride_w; p.dil_w = a.dil_w;
    p.N = a.N; p.P = a.P; p.Q = a.Q; p.Kout = a.Kout;
    const bool out_strided = (a.out_stride_w | a.out_stride_h | a.out_stride_n) != 0;
    p.o_sw = out_strided ? a.out_stride_w : a.Kout;
    p.o_sh = out_strided ? a.out_stride_h : (long long)a.Q * a.Kout;
    p.o_sn = out_strided ? a.out_stride_n : (long long)a.P * a.Q * a.Kout;
    p.act = a.act;
    // (not in the pooling instantiation: its epilogue has no registers to spare)
    p.split_acc = (p.issuers == 2 && 4 * p.MT * p.BN <= 512 && !a.pool_out && tune(TUNE_SPLIT_ACC, 1)) ? 1 : 0;
    p.tmem_cols = 32;
    while (p.tmem_cols < (p.split_acc ? 4 : 2) * p.MT * p.BN) p.tmem_cols *= 2;
    p.bias = a.bias; p.mask_src = a.mask_src; p.out = a.out;
    p.mask_mode = a.mask_mode; p.lr = a.lr;
    // split reduction: raw partial tiles to the caller's scratch, bias and activation after the splits are added
    p.ksplit = 1; p.kps = 0; p.split_stride = 0;
    if (a.split_ws) {
        int k = choose_ksplit(a, cfg, p.cblocks, g_sm_count);
        const size_t per = size_t(a.N) * a.P * a.Q * a.Kout * 4;
        while (k > 1 && (size_t(k) * per > a.split_ws_bytes || (a.R * a.S * p.cblocks / cfg.KS) % k != 0)) --k;
        if (k > 1 && m_tiles * p.tiles_k * k <= 0x7fffffffL) {
            p.ksplit = k; p.kps = a.R * a.S * p.cblocks / k; p.split_stride = per / 4;
            p.out = a.split_ws; p.bias = nullptr; p.act = PCL_ACT_NONE;
        }
    }
    if (a.pool_out && !tc_fprop_can_pool(a)) return PCL_ERR_UNSUPPORTED_SHAPE;
    p.pool_out = a.pool_out;
    p.pool_idx = a.pool_out ? a.pool_idx : nullptr;
    p.bias_in_smem = (a.pool_out && p.tiles_k == 1 && p.BN <= 256) ? 1 : 0;
    {
        const int slots = p.cblocks * ((a.R * a.S + cfg.KS - 1) / cfg.KS);
        p.resident_b = (cfg.halo && !cfg.pair && p.issuers == 1 && p.tiles_k == 1 && !p.bmn && slots <= 3 && slots <= cfg.stages &&      // (a launch keeps at least three slots)
                        tune(TUNE_RESIDENT_B, 1)) ? 1 : 0;
        p.kslices = (a.k_live > 0 && a.k_live < 32 && tune(TUNE_KSLICES, 1)) ? (a.k_live + 7) / 8 : 4;
        p.tile_duo = (p.resident_b && p.cblocks == 1 && p.NA % 2 == 0 && tune(TUNE_ISSUERS, 2) >= 2) ? 1 : 0;
    }
    p.colsum_rows = (a.Kout % 4 == 0) ? a.colsum_rows : nullptr;
    p.colsum_cta = (p.colsum_rows && p.tiles_k == 1 && p.ksplit == 1) ? 1 : 0;
    if (a.colsum_rows && !p.colsum_rows) return PCL_ERR_UNSUPPORTED_SHAPE;
    p.status = device_status_ptr();
    if (!p.status) return PCL_ERR_CUDA;
    // test mode (FAULT_INJECT knob = 1): only a non-pair launch in the plain tiling takes it
    p.inject_short_copy = (tune(TUNE_FAULT_INJECT, 0) == 1 && !cfg.pair && !cfg.halo) ? 1 : 0;

    CUtensorMap tmA, tmB;
    {
        const uint64_t dims[4] = {uint64_t(a.in_inner ? a.in_inner : a.Cin), uint64_t(a.W), uint64_t(a.H),
                                  uint64_t(a.N)};
        const uint64_t sw = a.in_stride_w ? uint64_t(a.in_stride_w) : uint64_t(a.Cin);
        const uint64_t sh = a.in_stride_h ? uint64_t(a.in_stride_h) : uint64_t(a.W) * a.Cin;
        const uint64_t sn = a.in_stride_n ? uint64_t(a.in_stride_n) : uint64_t(a.H) * a.W * a.Cin;
        const uint64_t strides[3] = {sw * 4, sh * 4, sn * 4};
        const uint32_t box_plain[4] = {kBlockC, uint32_t(bw * a.stride_w), uint32_t(bh * a.stride_h), uint32_t(bn)};
        const uint32_t estr[5] = {1, uint32_t(a.stride_w), uint32_t(a.stride_h), 1, 1};
        const uint32_t box_halo[4] = {kBlockC, uint32_t(p.PW), uint32_t(p.th + a.R - 1), 1};
        int rc;
        if (cfg.grp && !cfg.halo) {
            // channel blocks as a fifth dimension (128 bytes apart), so that one box spans KS of them
            const uint64_t dims5[5] = {kBlockC, uint64_t(a.W), uint64_t(a.H), uint64_t(a.N), uint64_t(p.cblocks)};
            const uint64_t strides5[4] = {sw * 4, sh * 4, sn * 4, kBlockC * 4};
            const uint32_t box5[5] = {kBlockC, uint32_t(bw * a.stride_w), uint32_t(bh * a.stride_h), uint32_t(bn), uint32_t(p.KS)};
            rc = make_tmap(&tmA, a.in, 5, dims5, strides5, box5, false, false, estr);
        } else {
            rc = make_tmap(&tmA, a.in, 4, dims, strides, p.halo ? box_halo : box_plain, false, false, p.halo ? nullptr : estr);
        }
        if (rc != PCL_OK) return rc;
    }
    {
        const uint64_t dims[3] = {uint64_t(a.Cin), uint64_t(a.R) * a.S, uint64_t(a.Kout)};
        const uint64_t strides[2] = {uint64_t(a.Cin) * 4, uint64_t(a.R) * a.S * a.Cin * 4};
        const uint32_t box[3] = {kBlockC, 1, uint32_t(cfg.pair ? p.BN / 2 : p.BN)};
        int rc;
        if (a.wt_mn_major) {
            // weights [Cin][R*S][Kout]: {32 maps, reduction rows, tap, 32-map group}; a box lands as
            // [group][32 (x KS in the plain tiling) reduction rows][32 maps], the MN-major operand layout
            const uint64_t dims4[4] = {kBlockC, uint64_t(a.Cin), uint64_t(a.R) * a.S, uint64_t(a.Kout / kBlockC)};
            const uint64_t strides4[3] = {uint64_t(a.R) * a.S * a.Kout * 4, uint64_t(a.Kout) * 4, kBlockC * 4};
            const uint32_t box4[4] = {kBlockC, uint32_t(kBlockC * ((cfg.grp && !cfg.halo) ? p.KS : 1)), 1,
                                      uint32_t((cfg.pair ? p.BN / 2 : p.BN) / kBlockC)};
            rc = make_tmap(&tmB, a.wt, 4, dims4, strides4, box4, true);
        } else if (cfg.grp && cfg.halo) {
            // {channel, output map, tap}: a box of KS taps lands as KS weight tiles
            const uint64_t dims3[3] = {uint64_t(a.Cin), uint64_t(a.Kout), uint64_t(a.R) * a.S};
            const uint64_t strides3[2] = {uint64_t(a.R) * a.S * a.Cin * 4, uint64_t(a.Cin) * 4};
            const uint32_t box3[3] = {kBlockC, uint32_t(cfg.pair ? p.BN / 2 : p.BN), uint32_t(p.KS)};
            rc = make_tmap(&tmB, a.wt, 3, dims3, strides3, box3, false);
        } else if (cfg.grp) {
            // {channel in block, output map, channel block, tap}: a box of KS channel blocks lands as KS weight tiles
            const uint64_t dims4[4] = {kBlockC, uint64_t(a.Kout), uint64_t(p.cblocks), uint64_t(a.R) * a.S};
            const uint64_t strides4[3] = {uint64_t(a.R) * a.S * a.Cin * 4, kBlockC * 4, uint64_t(a.Cin) * 4};
            const uint32_t box4[4] = {kBlockC, uint32_t(cfg.pair ? p.BN / 2 : p.BN), uint32_t(p.KS), 1};
            rc = make_tmap(&tmB, a.wt, 4, dims4, strides4, box4, false);
        } else {
            rc = make_tmap(&tmB, a.wt, 3, dims, strides, box, false);
        }
        if (rc != PCL_OK) return rc;
    }
    // Output map for the TMA-store epilogue: a warp stores the 32 consecutive box pixels it owns, 32 maps at a time.
    CUtensorMap tmOut = tmA;        // (a valid map is passed in any case; unused unless p.tma_store)
    p.tma_store = 0;
    if (p.ksplit > 1) {
        // (split partials go out through the per-lane path: plain stores at out + split * split_stride)
    } else if (!a.out) {
        // pooled output only: the epilogue stages each chunk as for a TMA store, takes the maxima from the staging
        // tile and stores nothing at full resolution
        if (!a.pool_out || a.colsum_rows) return PCL_ERR_BAD_ARG;
        p.tma_store = 1;
    } else if (tune(TUNE_TMA_STORE, 1) && !out_strided && !a.mask_src && !a.colsum_rows && a.Kout % 4 == 0 &&
        (reinterpret_cast<uintptr_t>(a.out) & 15) == 0) {
        const uint32_t bx = bw < 32 ? bw : 32, by = uint32_t(bh) < 32 / bx ? uint32_t(bh) : 32 / bx, bnn = 32 / (bx * by);
        const uint64_t dims[4] = {uint64_t(a.Kout), uint64_t(a.Q), uint64_t(a.P), uint64_t(a.N)};
        const uint64_t strides[3] = {uint64_t(a.Kout) * 4, uint64_t(a.Q) * a.Kout * 4, uint64_t(a.P) * a.Q * a.Kout * 4};
        const uint32_t box[4] = {kBlockC, bx, by, bnn};
        if (make_tmap(&tmOut, a.out, 4, dims, strides, box, false, true) == PCL_OK) p.tma_store = 1;
        else tmOut = tmA;
    }
    // Sixteen epilogue warps where the epilogue bounds the tile: estimated cycles of a box's MMAs (a K8 step of
    // BN <= 64 columns takes ~50 cycles, wider ones BN/2) against ~1600 cycles per 32-column chunk and warp.  Their
    // staging tiles take 32 KB more; the ring gives up slots for them as long as three remain.
    bool wide_epi = false;
    const int epi_hook = tune(TUNE_EPI_WARPS, 16);      // test hook: 8 = never, 32 = wherever the variant can run
    if (!cfg.pair && p.tma_store && !p.split_acc && epi_hook >= 16) {
        const long mma_clk = long(a.R) * a.S * p.cblocks * 4 * (p.BN <= 64 ? 50 : p.BN / 2);
        const long epi_clk = long(p.BN / 32) * 1600 / 2;
        if (2 * epi_clk > 3 * mma_clk || epi_hook >= 32) {
            const int slot = p.KS * (p.halo ? p.BN * 128 : kABytes + p.BN * 128);
            const int fixed = (p.halo ? p.NA * p.a_buf_bytes : 0) + kEpiStageBytesWide;
            int stages = p.stages;
            while (stages > 3 && fixed + stages * slot > kSmemBudget) --stages;
            if (fixed + stages * slot <= kSmemBudget) { p.stages = stages; wide_epi = true; }
        }
    }
    const long total = m_tiles * p.tiles_k * p.ksplit;
    const size_t smem = (p.halo ? size_t(p.NA) * p.a_buf_bytes + size_t(p.stages) * p.KS * (cfg.pair ? p.BN * 64 : p.BN * 128)
                                : size_t(p.stages) * p.KS * (kABytes + (cfg.pair ? p.BN * 64 : p.BN * 128))) +
                        (wide_epi ? kEpiStageBytesWide : kEpiStageBytes) + 1024;
    plan->p = p; plan->tmA = tmA; plan->tmB = tmB; plan->tmOut = tmOut;
    plan->pair = cfg.pair != 0; plan->wide_epi = wide_epi; plan->smem = smem; plan->total = total; plan->sm_count = g_sm_count;
    plan->flops = 2.0 * a.N * a.P * a.Q * double(a.Kout) * a.Cin * a.R * a.S;
    plan->grid = int(total < g_sm_count ? total : g_sm_count);
    if (cfg.pair) {
        // how many pairs the device holds at once with this much shared memory (cached per size)
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t lc{};
        lc.blockDim = dim3(kThreads); lc.dynamicSmemBytes = smem;
        lc.attrs = attr; lc.numAttrs = 1;
        static std::mutex cache_mu;
        static size_t cached_smem = 0;
        static int cached_clusters = 0, cached_dev = -1;
        int cur_dev = 0;
        if (cudaGetDevice(&cur_dev) != cudaSuccess) return PCL_ERR_CUDA;
        std::lock_guard<std::mutex> cache_lock(cache_mu);
        if (cached_smem != smem || cached_dev != cur_dev) {
            lc.gridDim = dim3(unsigned(g_sm_count / 2 * 2));
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, tc_fprop_kernel<true, false, false>, &lc) != cudaSuccess || n <= 0) return PCL_ERR_CUDA;
            cached_clusters = n < g_sm_count / 2 ? n : g_sm_count / 2;
            cached_smem = smem;
            cached_dev = cur_dev;
        }
        const long nclus = total < cached_clusters ? total : cached_clusters;       // (total counts pair tiles here)
        plan->grid = int(2 * nclus);
    }
    return PCL_OK;
}

int run_fprop_plan(const FpropPlan& plan, const TcFpropArgs& a, cudaStream_t st) {
    const FpropParams& p = plan.p;
    const CUtensorMap& tmA = plan.tmA;
    const CUtensorMap& tmB = plan.tmB;
    const CUtensorMap& tmOut = plan.tmOut;
    const bool wide_epi = plan.wide_epi;
    const size_t smem = plan.smem;
    if (plan.pair) {
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t lc{};
        lc.blockDim = dim3(kThreads); lc.dynamicSmemBytes = smem; lc.stream = st;
        lc.attrs = attr; lc.numAttrs = 1;
        lc.gridDim = dim3(unsigned(plan.grid));
        LaunchScope scope(KID_TC_FPROP, plan.flops, st);
        const cudaError_t le = p.pool_out   ? cudaLaunchKernelEx(&lc, tc_fprop_kernel<true, true, false>, tmA, tmB, tmOut, p)
                               : p.mask_src ? cudaLaunchKernelEx(&lc, tc_fprop_kernel<true, false, true>, tmA, tmB, tmOut, p)
                                            : cudaLaunchKernelEx(&lc, tc_fprop_kernel<true, false, false>, tmA, tmB, tmOut, p);
        if (le != cudaSuccess) return PCL_ERR_CUDA;
    } else {
        const int grid = plan.grid;
        LaunchScope scope(KID_TC_FPROP, plan.flops, st);
        if (wide_epi && p.pool_out) tc_fprop_kernel<false, true, false, kEpiWarpsWide><<<grid, kThreadsWide, smem, st>>>(tmA, tmB, tmOut, p);
        else if (wide_epi) tc_fprop_kernel<false, false, false, kEpiWarpsWide><<<grid, kThreadsWide, smem, st>>>(tmA, tmB, tmOut, p);
        else if (p.pool_out) tc_fprop_kernel<false, true, false><<<grid, kThreads, smem, st>>>(tmA, tmB, tmOut, p);
        else if (p.mask_src) tc_fprop_kernel<false, false, true><<<grid, kThreads, smem, st>>>(tmA, tmB, tmOut, p);
        else tc_fprop_kernel<false, false, false><<<grid, kThreads, smem, st>>>(tmA, tmB, tmOut, p);
    }
    if (cudaGetLastError() != cudaSuccess) return PCL_ERR_CUDA;
    if (p.ksplit > 1)
        return launch_reduce_splits_bias_act(a.split_ws, a.out, a.bias, a.act, size_t(a.N) * a.P * a.Q, a.Kout, p.ksplit, st);
    return PCL_OK;
}
}  // namespace

}  // namespace pcl
