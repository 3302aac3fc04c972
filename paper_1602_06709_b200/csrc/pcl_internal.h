// Internal launcher interfaces shared by the .cu files of the library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/pcl_dnn.h"

namespace pcl {

#ifdef __CUDACC__
// Logistic function from the two approximate special-function instructions (ex2 and rcp, each within 2 ulp): an
// IEEE division per element costs a one-tile GEMM's epilogue several microseconds.
__device__ __forceinline__ float sigmoid_fast(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }
#endif

// Kernel families, for launch counting and the optional per-kernel timing.
enum KernelId {
    KID_TC_FPROP = 0, KID_TC_WGRAD, KID_GENERIC_FWD, KID_GENERIC_DGRAD, KID_GENERIC_WGRAD, KID_SGD, KID_REDUCE_SPLITS,
    KID_ZERO, KID_TRANSPOSE_FLIP, KID_ACT_GRAD, KID_COLSUM, KID_MAXPOOL_FWD, KID_MAXPOOL_BWD, KID_SOFTMAX_XENT,
    KID_STAGE_PAD_C4, KID_STAGE_W4, KID_UNPAD_REDUCE, KID_COUNT
};

// Brackets one kernel launch: counts it and, while profiling is switched on
// (pcl_profile_begin), records a CUDA event on the launching stream before and
// after it.  `work` is the launch's algorithmic work: flops for the contraction
// kernels, bytes for the memory-bound ones.
struct LaunchScope {
    LaunchScope(int kid, double work, cudaStream_t st);
    ~LaunchScope();
    LaunchScope(const LaunchScope&) = delete;
    LaunchScope& operator=(const LaunchScope&) = delete;
    int slot;
    cudaStream_t st;
};

// Tags the launches an ABI call makes with the pass they belong to (for the per-pass timing of pcl_profile_end) and
// carries the layer's own algorithmic flops for its contraction launches.  Nested calls keep the outermost tag.
enum ProfPass { PROF_PASS_OTHER = 0, PROF_PASS_CONV_FWD, PROF_PASS_CONV_BWD_DATA, PROF_PASS_CONV_BWD_WEIGHTS,
                PROF_PASS_FC_FWD, PROF_PASS_FC_BWD, PROF_PASS_COUNT };
struct PassScope {
    PassScope(int pass, double flops, int contraction_launches = 1);
    ~PassScope();
    PassScope(const PassScope&) = delete;
    PassScope& operator=(const PassScope&) = delete;
};
double conv_pass_flops(const pcl_conv_desc& d, int P, int Q);
// Mandatory part of the backward-data workspace: bytes of the transposed weight copy, 0 where none is made.
size_t bwd_data_transposed_bytes(const pcl_conv_desc& d);

// Test / tuning knobs: every choice the launchers make has one, so that the tests can pin each pipeline variant and
// the alternatives can be measured.  They are set through pcl_set_tuning() only (never read from the environment:
// a stray variable must not change which kernel a production call runs); tune() returns the knob's value, or
// `dflt` while it is unset.
enum TuneId {
    TUNE_TILING = 0,        // forward-type kernel: 0 plain, 1-3 haloed layouts 0-2
    TUNE_BN, TUNE_KS, TUNE_KS_HALO, TUNE_KS_WGRAD, TUNE_PAIR, TUNE_PAIR_HALO, TUNE_PAIR_WGRAD, TUNE_GRP, TUNE_ISSUERS,
    TUNE_SPLIT_ACC, TUNE_PIX_WGRAD, TUNE_XHALO_WGRAD, TUNE_TMA_STORE, TUNE_WEIGHTS_IN_PLACE, TUNE_EPI_WARPS,
    TUNE_FC_DW_FORWARD, TUNE_KSPLIT, TUNE_WAIT_LIMIT_US, TUNE_FAULT_INJECT, TUNE_RESIDENT_B, TUNE_KSLICES, TUNE_SELECT, TUNE_PACKED_BWD, TUNE_PLAN_CACHE, TUNE_COUNT
};
int tune(int id, int dflt);
bool tune_is_set(int id);
unsigned tune_generation();      // bumped by every pcl_set_tuning / pcl_reset_tuning (cached launch plans key on it)

// SM count of the current device (cached per device, thread-safe).  Without a usable device (a sizing query on a
// machine that has none) the B200's 148 is returned: a launch would fail there anyway.
int device_sm_count();
// Runs `setup` once per device (thread-safe) and remembers its success; used for cudaFuncSetAttribute, which
// applies to the current device only.
struct PerDeviceOnce {
    template <class F>
    int run(F&& setup) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PCL_ERR_CUDA;
        if (done_[dev].load(std::memory_order_acquire)) return PCL_OK;
        std::lock_guard<std::mutex> lock(mu_);
        if (done_[dev].load(std::memory_order_relaxed)) return PCL_OK;
        const int rc = setup();
        if (rc == PCL_OK) done_[dev].store(true, std::memory_order_release);
        return rc;
    }
  private:
    std::mutex mu_;
    std::atomic<bool> done_[64] = {};
};

// Device status word values that are not wait codes (those are 0x1xx, see pcl_ptx.cuh).
constexpr unsigned int kStatusBadLabel = 0x201;     // pcl_softmax_xent met a label outside [0, K)

// Address of the current device's status word (0 = fine, else the code of the
// first bounded wait that ran out).  nullptr if the address cannot be obtained.
unsigned int* device_status_ptr();

// Driver entry point for cuTensorMapEncodeTiled, fetched at run time so that the
// library has no link-time dependency on libcuda.  Returns nullptr on failure.
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
encode_tiled_fn get_encode_tiled();

// fp32 tensor map with a 128-byte swizzle span, swizzled in 16-byte chunks
// (K-major operands) or, if atom32, in 32-byte chunks (MN-major operands).
// dims/box innermost first; strides_bytes has rank-1 entries (dims 1..rank-1).
// The element type is TFLOAT32 (TMA rounds fp32 to tf32, nearest-even, on load) unless plain_f32 (maps used for stores).
// elem_strides (optional, rank entries): traversal stride per dimension; a dimension with stride t > 1 takes every
// t-th element, and its box entry counts elements of the tensor (box / t elements land in shared memory).
int make_tmap(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box, bool atom32, bool plain_f32 = false, const uint32_t* elem_strides = nullptr);

// ---- forward-type implicit GEMM on tcgen05 -----------------------------------
// out[n,p,q,k] = epi( sum_{r,s,c} in[n, p*stride_h + r - pad_h, q*stride_w + s*dil_w - pad_w, c] * wt[k, r*S+s, c] )
// epi: + bias[k], activation, optional zeroing where mask_src[n,p,q,k] <= 0.
struct TcFpropArgs {
    const float* in;   // [N][H][W][Cin]
    const float* wt;   // [Kout][R*S][Cin]
    const float* bias; // [Kout] or null
    const float* mask_src; // [N][P][Q][Kout] or null (see mask_mode)
    float* out;        // [N][P][Q][Kout]; may be null with pool_out (nothing is stored at full resolution)
    int N, H, W, Cin, Kout, R, S, pad_h, pad_w, P, Q, act;
    // Element strides of `in` between adjacent w, h and n positions; 0 = packed
    // NHWC (Cin, W*Cin, H*W*Cin).  A w stride smaller than Cin gives overlapping
    // windows (used by the few-channel first-layer path).
    long in_stride_w = 0, in_stride_h = 0, in_stride_n = 0;
    // What mask_src does: 0 = the output is zeroed where mask_src <= 0 (gradient of the ReLU that produced mask_src);
    // 1 = the output is multiplied by mask_src * (1 - mask_src) (gradient of the sigmoid that produced mask_src).
    int mask_mode = 0;
    float lr = 0.f;         // mask_mode 2: out = mask_src - lr * (the contraction); out may be mask_src itself (SGD in place)
    // k_live (0 = all): how many leading elements of every 32-element channel block can be non-zero in `wt` (the
    // few-channel path packs S taps x 4 channels into a block and zero-fills the rest): MMAs over all-zero K = 8
    // slices are skipped.
    int k_live = 0;
    // Innermost extent the tensor map declares (0 = Cin).  The few-channel path declares 32 although only Cin
    // elements carry weight: the rest of the window is real neighbouring data that meets zero weights, which
    // avoids TMA's slower partial-row zero fill.
    int in_inner = 0;
    // Optional fused column sums of the output (after bias / activation / mask), Kout % 4 == 0: rows of per-column
    // sums go to `colsum_rows` -- one per (CTA, tile box, 32-row quarter) when all tiles have the same columns (the
    // sums are kept over the CTA's tiles), else one per (tile, box, quarter); tc_fprop_colsum_rows_written(a) rows,
    // of which a small grid may leave some untouched (zero them first); the caller adds the rows in a fixed order.
    float* colsum_rows = nullptr;
    // Optional fused 2x2 / stride-2 max pooling of the output: pool_out [N][P/2][Q/2][Kout] gets the window maxima
    // of `out` (after bias and activation).  Needs even P and Q and Kout % 4 == 0 (tc_fprop_can_pool()).
    float* pool_out = nullptr;
    // with pool_out: [N][P/2][Q/2][Kout] bytes, bits 0-1 = position of the window's first maximum (row-major), bit 2 set
    // where that maximum is <= 0 (what a ReLU mask would zero); lets the pooling backward pass skip reading `out`
    unsigned char* pool_idx = nullptr;
    // Optional scratch for a split reduction (launches with few tiles and a long reduction): if given, and the
    // launcher finds splits worth while and the scratch large enough (tc_fprop_split_ws_bytes()), every split's raw
    // partial tile goes there and a second pass adds them in a fixed order and applies bias and activation.
    float* split_ws = nullptr;
    size_t split_ws_bytes = 0;
    // wt_mn_major != 0: `wt` is laid out [Cin][R*S][Kout] (output maps innermost), i.e. a layer's own KRSC weights
    // seen from its backward-data pass (reduction over the layer's K, columns = the layer's C): the kernel then
    // reads B as an MN-major operand and no transposed copy is needed.  Needs Kout % 32 == 0.
    // flip_taps != 0: tap t of the loop reads tap R*S-1-t of `wt` (the spatial flip of backward-data).
    int wt_mn_major = 0, flip_taps = 0;
    // Strides of the convolution (fetched by TMA with a traversal stride: only the pixels a tile needs are read) and
    // the distance in pixels between consecutive taps of a kernel row (8 on the few-channel path when a kernel row
    // is wider than one 32-float window: tap s' then covers kernel columns 8s' .. 8s'+7).  pad_h / pad_w may be
    // negative (the phases of a strided backward-data pass).
    int stride_h = 1, stride_w = 1, dil_w = 1;
    // Element strides of `out` (and of mask_src) between adjacent q, p and n positions; 0 = packed NPQK.  A strided
    // backward-data pass writes each of its phases to every stride-th pixel of dx.
    long out_stride_w = 0, out_stride_h = 0, out_stride_n = 0;
};
bool tc_fprop_can_pool(const TcFpropArgs& a);
// bytes of split_ws with which launch_tc_fprop(a) would split the reduction (0: it would not)
size_t tc_fprop_split_ws_bytes(const TcFpropArgs& a);
bool tc_fprop_eligible(const TcFpropArgs& a);
long tc_fprop_colsum_rows(const TcFpropArgs& a);              // upper bound over all tilings (workspace sizing)
// rows the launch for exactly these arguments writes (rows 0 .. n-1); *all_written: none of them is left untouched
long tc_fprop_colsum_rows_written(const TcFpropArgs& a, bool* all_written = nullptr);
int launch_tc_fprop(const TcFpropArgs& a, cudaStream_t st);
// tensor-core launches whose plan (tiling, kernel parameters, tensor maps, grid) came out of / went into the plan caches
void plan_cache_count(bool hit);
void plan_cache_stats(unsigned long long* hits, unsigned long long* misses);
// Text description of the tiling launch_tc_fprop(a) would use and of the cost model's prediction for it (and of the
// tiling the model itself would choose).
int tc_fprop_describe(const TcFpropArgs& a, char* buf, size_t n);

// ---- weight-gradient-type GEMM on tcgen05 ------------------------------------
// dw[k, r, s, c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride_h + r - pad_h, q*stride_w + s*dil_w - pad_w, c]
struct TcWgradArgs {
    const float* x;   // [N][H][W][C]
    const float* dy;  // [N][P][Q][K]
    float* dw;        // [K][R][S][C]
    float* partial;   // workspace for the two-pass variant ([splits][K*R*S*C]) or null (atomics)
    int N, H, W, C, K, R, S, pad_h, pad_w, P, Q;
    int splits;
    // Element strides of x (0 = packed NHWC), as in TcFpropArgs.
    long x_stride_w = 0, x_stride_h = 0, x_stride_n = 0;
    int x_inner = 0;   // innermost extent declared for x (0 = C); see TcFpropArgs::in_inner
    // tap_groups != 0: S must be 1 and C <= 32; one CTA handles all R taps of a k
    // tile at once, the MMA N dimension being R groups of 32 columns (group g =
    // tap row g).  dw then has the layout [K][R][C].
    int tap_groups = 0;
    // skip_reduce != 0: leave the per-split partial tiles in `partial` (the caller reduces them).
    int skip_reduce = 0;
    // Pooled dy: `dy` is null and the kernel builds its dy tiles from dy_pool [N][P/2][Q/2][K] and the pooling
    // windows' position codes (same shape, bytes): the coded position of each window gets the gradient, the other
    // three zero; relu_mask: windows whose code has bit 2 set get nothing.  db_rows (optional, [splits * kPooledDbRows][K]) gets
    // per-(split, epilogue warp) sums of the scattered gradient, i.e. the bias gradient before the rows are added.
    // Needs even P and Q, K % 4 == 0, single-CTA items (tc_wgrad_can_take_pooled_dy()).
    const float* dy_pool = nullptr;
    const unsigned char* codes = nullptr;
    int relu_mask = 0;
    float* db_rows = nullptr;
    int stride_h = 1, stride_w = 1, dil_w = 1;      // as in TcFpropArgs
    // unsplit launches (splits == 1): instead of storing dw the epilogue writes w_update[i] - lr * dw[i] in place
    float* w_update = nullptr;
    float lr = 0.f;
};
bool tc_wgrad_eligible(const TcWgradArgs& a);
constexpr int kPooledDbRows = 16;       // bias-gradient rows per pixel split that a pooled-dy launch writes
bool tc_wgrad_can_take_pooled_dy(int N, int P, int Q, int C, int K, int R, int S, int tap_groups);
int tc_wgrad_splits(int N, int P, int Q, int C, int K, int R, int S, int tap_groups = 0, int pooled_dy = 0,
                    int strided = 0);
int launch_tc_wgrad(const TcWgradArgs& a, cudaStream_t st);

// ---- generic CUDA-core kernels (any stride / pad / channel count) ----------
int launch_generic_fwd(const pcl_conv_desc& d, int P, int Q, const float* x, const float* w, const float* bias,
                       float* y, int act, cudaStream_t st);
int launch_generic_bwd_data(const pcl_conv_desc& d, int P, int Q, const float* dy, const float* w,
                            const float* mask_src, float* dx, cudaStream_t st);
int generic_wgrad_splits(const pcl_conv_desc& d, int P, int Q);
int launch_generic_bwd_weights(const pcl_conv_desc& d, int P, int Q, const float* x, const float* dy, float* dw,
                               float* partial, int splits, cudaStream_t st);

// ---- HBM-bound helpers ------------------------------------------------------
int launch_sgd(float* w, const float* dw, size_t n, float lr, cudaStream_t st);
int launch_reduce_splits(const float* partial, float* out, size_t n, int splits, cudaStream_t st);
int launch_reduce_splits_sgd(const float* partial, float* w, size_t n, int splits, float lr, cudaStream_t st);
// out[r][k] = act(bias[k] + sum_s partial[s][r][k]), splits added in index order; K % 4 == 0
int launch_reduce_splits_bias_act(const float* partial, float* out, const float* bias, int act, size_t rows, int K,
                                  int splits, cudaStream_t st);
int launch_zero(float* p, size_t n, cudaStream_t st);
// wt_t[c][R-1-r][S-1-s][k] = w[k][r][s][c]
int launch_transpose_flip(const float* w, float* wt_t, int K, int R, int S, int C, cudaStream_t st);
// One phase of a strided backward-data pass: wt_t[c][Ra-1-i][Sb-1-j][k] = w[k][a + i*stride_h][b + j*stride_w][c],
// i < Ra, j < Sb (the taps that reach input pixels of phase (a, b), flipped and transposed).
int launch_phase_weights(const float* w, float* wt_t, int K, int R, int S, int C, int a, int b, int stride_h,
                         int stride_w, int Ra, int Sb, cudaStream_t st);
// Phase-packed backward-data (strided layers with stride_h * stride_w * C <= 256): the sub-kernels of all phases as the
// output maps of ONE stride-1 convolution (wpk[col][Rm][Sm][K], col = (a*sw + b)*C + c, zero where a phase has no such
// tap), and the scatter of its output t[N][U][V][cols4] to dx (optionally zeroed where mask <= 0).
int launch_phase_pack_weights(const float* w, float* wpk, int K, int R, int S, int C, int sh, int sw, int Rm, int Sm,
                              int cols4, cudaStream_t st);
int launch_phase_unpack(const float* t, const float* mask, float* dx, int N, int H, int W, int C, int sh, int sw, int pad_h,
                        int pad_w, int U, int V, int cols4, cudaStream_t st);
// Few-channel staging (C < 4): xs[n][h+pad_h][w+pad_w][0..3] = x[n][h][w][0..C-1] padded with zeros (channel
// padding and a spatial halo of pad_h / pad_w), followed by `slack_pixels` zero pixels; w32[row][s*4 + c] =
// w[row][s][c] (row = k*R + r) in zero-padded rows of row_floats (a multiple of 32) floats;
// dw[row][s][c] = sum over splits of dw4[split][row][s*4 + c] with rows of row_floats floats.
int launch_stage_pad_c4(const float* x, float* xs, int N, int H, int W, int C, int pad_h, int pad_w, int slack_pixels,
                        cudaStream_t st);
int launch_stage_w4(const float* w, float* w32, size_t rows, int S, int C, int row_floats, cudaStream_t st);
int launch_unpad_reduce(const float* dw4, float* dw, size_t rows, int S, int C, int row_floats, int splits,
                        size_t split_stride, cudaStream_t st);
// dz = dy * act'(y), in place on dy
int launch_act_grad(float* dy, const float* y, size_t n, int act, cudaStream_t st);
// out[k] = sum_rows m[row][k]; partial: [colsum_splits(rows)][K] workspace
int colsum_splits(size_t rows);
int launch_colsum(const float* m, size_t rows, int K, float* partial, float* out, cudaStream_t st);
// idx (optional): per output the position code of its window (bits 0-1 first maximum, bit 2: maximum <= 0)
int launch_maxpool_fwd(int N, int H, int W, int C, const float* x, float* y, cudaStream_t st, unsigned char* idx = nullptr);
int launch_maxpool_bwd_idx(int N, int H, int W, int C, const unsigned char* idx, const float* dy, int relu, float* dx,
                           float* colsum_rows, cudaStream_t st);
int launch_maxpool_bwd(int N, int H, int W, int C, const float* x, const float* dy, const float* mask, float* dx,
                       cudaStream_t st);
// The same with fused per-block column sums of dx: colsum_rows is [maxpool_bwd_colsum_rows(N,H,W,C)][C]; returns 0
// rows when the shape cannot take the fused form (then use launch_colsum on dx).
long maxpool_bwd_colsum_rows(int N, int H, int W, int C);
int launch_maxpool_bwd_colsum(int N, int H, int W, int C, const float* x, const float* dy, const float* mask,
                              float* dx, float* colsum_rows, cudaStream_t st);
int launch_softmax_xent(int N, int K, const float* logits, const int* labels, float* loss, float* dlogits,
                        cudaStream_t st);

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace pcl
