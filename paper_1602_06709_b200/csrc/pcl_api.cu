// C ABI of the library: argument checks, kernel-family selection, workspace
// carving, tensor-map construction.  Every entry point only enqueues kernels on
// the caller's stream.
#include <atomic>
#include <mutex>
#include <limits.h>
#include <stdio.h>
#include <string.h>
#include <vector>

#include "pcl_internal.h"
#include "pcl_ptx.cuh"

namespace pcl {

// [0]: status word (0 = fine, else the code of the first bounded wait that ran out, or kStatusBadLabel);
// [1]: limit of the bounded device-side waits in microseconds
__device__ unsigned int g_device_status[2] = {0u, 2000000u};

unsigned int* device_status_ptr() {
    // one copy of the symbol per device: look the address up per device, once
    static unsigned int* cache[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<unsigned int*>(p);
    }
    return cache[dev];
}

static std::atomic<unsigned long long> g_launches{0};

namespace {
struct TuneSlot { std::atomic<int> set{0}; std::atomic<int> value{0}; };
TuneSlot g_tune[TUNE_COUNT];
std::atomic<unsigned> g_tune_gen{0};
const char* const kTuneNames[TUNE_COUNT] = {
    "TILING", "BN", "KS", "KS_HALO", "KS_WGRAD", "PAIR", "PAIR_HALO", "PAIR_WGRAD", "GRP", "ISSUERS", "SPLIT_ACC",
    "PIX_WGRAD", "XHALO_WGRAD", "TMA_STORE", "WEIGHTS_IN_PLACE", "EPI_WARPS", "FC_DW_FORWARD", "KSPLIT",
    "WAIT_LIMIT_US", "FAULT_INJECT", "RESIDENT_B", "KSLICES", "SELECT", "PACKED_BWD", "PLAN_CACHE"};
}  // namespace

int tune(int id, int dflt) {
    return g_tune[id].set.load(std::memory_order_relaxed) ? g_tune[id].value.load(std::memory_order_relaxed) : dflt;
}
bool tune_is_set(int id) { return g_tune[id].set.load(std::memory_order_relaxed) != 0; }
unsigned tune_generation() { return g_tune_gen.load(std::memory_order_relaxed); }

int device_sm_count() {
    static std::atomic<int> cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    cache[dev].store(n, std::memory_order_relaxed);
    return n;
}

namespace {
struct ProfEntry { int kid; int pass; double work; cudaEvent_t e0, e1; };
// Which ABI call the launches of this thread belong to (outermost call wins), and, for its contraction launches,
// the layer's own algorithmic work 2*N*K*P*Q*C*R*S: a launch that runs on a padded or staged view of the layer
// (few-channel staging, phase-decomposed strides) must not count the zero padding as work.
struct PassState { int pass = 0; int depth = 0; double flops = 0.0; int counted = 0; };
thread_local PassState t_pass;
const char* const kPassNames[PROF_PASS_COUNT] = {"other", "conv_fwd", "conv_bwd_data", "conv_bwd_weights", "fc_fwd", "fc_bwd"};
bool is_contraction(int kid) {
    return kid == KID_TC_FPROP || kid == KID_TC_WGRAD || kid == KID_GENERIC_FWD || kid == KID_GENERIC_DGRAD ||
           kid == KID_GENERIC_WGRAD;
}
std::mutex g_prof_mu;
bool g_prof_on = false;
std::vector<ProfEntry> g_prof_entries;       // entries of the current profiling window
std::vector<cudaEvent_t> g_prof_pool;        // events created so far, reused across windows
size_t g_prof_pool_used = 0;
const char* const kKernelNames[KID_COUNT] = {
    "tc_fprop_kernel", "tc_wgrad_kernel", "generic_fwd", "generic_bwd_data", "generic_bwd_weights", "sgd_kernel",
    "reduce_splits_kernel", "zero_kernel", "transpose_flip_kernel", "act_grad_kernel", "colsum_kernel",
    "maxpool_fwd_kernel", "maxpool_bwd_kernel", "softmax_xent_kernel", "stage_pad_c4_kernel", "stage_w4_kernel",
    "unpad_reduce_kernel"};

cudaEvent_t prof_event() {
    if (g_prof_pool_used == g_prof_pool.size()) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        g_prof_pool.push_back(e);
    }
    return g_prof_pool[g_prof_pool_used++];
}
}  // namespace

LaunchScope::LaunchScope(int kid, double work, cudaStream_t stream) : slot(-1), st(stream) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    std::lock_guard<std::mutex> lock(g_prof_mu);
    if (!g_prof_on) return;
    if (t_pass.depth > 0 && t_pass.flops > 0.0 && is_contraction(kid)) {
        // the first `counted` contraction launches of the call carry the layer's flops; a call that cuts one pass
        // into several launches (the phases of a strided backward-data pass) counts it once
        work = t_pass.counted > 0 ? t_pass.flops : 0.0;
        if (t_pass.counted > 0) --t_pass.counted;
    }
    ProfEntry e{kid, t_pass.depth > 0 ? t_pass.pass : PROF_PASS_OTHER, work, prof_event(), prof_event()};
    if (!e.e0 || !e.e1) return;
    cudaEventRecord(e.e0, st);
    slot = int(g_prof_entries.size());
    g_prof_entries.push_back(e);
}

LaunchScope::~LaunchScope() {
    if (slot < 0) return;
    std::lock_guard<std::mutex> lock(g_prof_mu);
    if (slot < int(g_prof_entries.size())) cudaEventRecord(g_prof_entries[slot].e1, st);
}

PassScope::PassScope(int pass, double flops, int contraction_launches) {
    if (t_pass.depth++ == 0) { t_pass.pass = pass; t_pass.flops = flops; t_pass.counted = contraction_launches; }
}
PassScope::~PassScope() {
    if (--t_pass.depth == 0) { t_pass.pass = PROF_PASS_OTHER; t_pass.flops = 0.0; }
}
double conv_pass_flops(const pcl_conv_desc& d, int P, int Q) {
    return 2.0 * d.N * double(d.K) * P * Q * double(d.C) * d.R * d.S;
}

static std::atomic<int> g_path{PCL_PATH_AUTO};

encode_tiled_fn get_encode_tiled() {
    static encode_tiled_fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(p);
    });
    return fn;
}

int make_tmap(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box, bool atom32, bool plain_f32, const uint32_t* elem_strides) {
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return PCL_ERR_CUDA;
    cuuint64_t gdim[5];
    cuuint64_t gstr[4];
    cuuint32_t gbox[5], estr[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        gbox[i] = box[i];
        estr[i] = elem_strides ? elem_strides[i] : 1;
        if (box[i] == 0 || box[i] > 256 || estr[i] == 0 || estr[i] > 8) return PCL_ERR_UNSUPPORTED_SHAPE;
    }
    for (int i = 0; i + 1 < rank; ++i) {
        gstr[i] = strides_bytes[i];
        if (strides_bytes[i] % 16 != 0 || strides_bytes[i] >= (1ull << 40)) return PCL_ERR_UNSUPPORTED_SHAPE;
    }
    if (reinterpret_cast<uintptr_t>(base) & 15) return PCL_ERR_MISALIGNED;
    const CUresult r = enc(out, plain_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, cuuint32_t(rank), const_cast<void*>(base), gdim, gstr,
                           gbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PCL_OK : PCL_ERR_CUDA;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Backward-data on the tensor-core path reads the KRSC weights in place (as an MN-major operand) when the layer's
// input-map count is a multiple of 32; otherwise it goes through a flipped, transposed copy in the workspace.
// The WEIGHTS_IN_PLACE knob set to 0 forces the copy (test hook).
bool weights_read_in_place(const pcl_conv_desc& d) { return d.C % 32 == 0 && tune(TUNE_WEIGHTS_IN_PLACE, 1) != 0; }

size_t dw_bytes(const pcl_conv_desc& d);
// Backward-data of a strided layer whose stride_h * stride_w * C fits one tile width runs as ONE stride-1 convolution
// whose output maps are (phase, input map) pairs, plus a scatter of that output to dx; wider layers run one launch per
// phase (conv_bwd_data_phases).
struct StridedBwdPlan { bool packed; int Rm, Sm, U, V, cols4; size_t wpk_bytes, temp_bytes; };
StridedBwdPlan strided_bwd_plan(const pcl_conv_desc& d) {
    StridedBwdPlan p{};
    const int cols = d.stride_h * d.stride_w * d.C;
    p.cols4 = (cols + 3) / 4 * 4;
    p.Rm = (d.R + d.stride_h - 1) / d.stride_h; p.Sm = (d.S + d.stride_w - 1) / d.stride_w;
    p.U = (d.H - 1 + d.pad_h) / d.stride_h + 1; p.V = (d.W - 1 + d.pad_w) / d.stride_w + 1;
    p.packed = p.cols4 <= 256 && d.K % 4 == 0;
    p.wpk_bytes = align_up(size_t(p.cols4) * p.Rm * p.Sm * d.K * 4, 256);
    p.temp_bytes = align_up(size_t(d.N) * p.U * p.V * p.cols4 * 4, 256);
    return p;
}
}  // namespace

// Bytes of the flipped, transposed weight copy backward-data makes on the tensor-core path (0 where the weights
// are read in place or another kernel family runs): the part of the backward-data workspace that is mandatory.
size_t bwd_data_transposed_bytes(const pcl_conv_desc& d) {
    if (g_path.load() == PCL_PATH_GENERIC || d.K % 4 != 0) return 0;
    if (d.stride_h != 1 || d.stride_w != 1) {
        if (d.stride_h > 8 || d.stride_w > 8) return 0;
        const StridedBwdPlan sp = strided_bwd_plan(d);
        const size_t phases = dw_bytes(d) + size_t(256) * d.stride_h * d.stride_w;    // one flipped, transposed sub-kernel per phase, 256-byte aligned
        const size_t packed = sp.wpk_bytes + sp.temp_bytes;
        return sp.packed && packed > phases ? packed : phases;
    }
    if (!(d.pad_h <= d.R - 1 && d.pad_w <= d.S - 1)) return 0;
    return weights_read_in_place(d) ? 0 : dw_bytes(d);
}

namespace {
int check_desc(const pcl_conv_desc* d, int* P, int* Q) {
    if (!d) return PCL_ERR_BAD_ARG;
    if (d->N <= 0 || d->C <= 0 || d->K <= 0 || d->H <= 0 || d->W <= 0 || d->R <= 0 || d->S <= 0 || d->stride_h <= 0 ||
        d->stride_w <= 0 || d->pad_h < 0 || d->pad_w < 0)
        return PCL_ERR_BAD_ARG;
    const long sh = long(d->H) + 2L * d->pad_h - d->R, sw = long(d->W) + 2L * d->pad_w - d->S;
    if (sh < 0 || sw < 0) return PCL_ERR_BAD_ARG;
    *P = int(sh / d->stride_h) + 1;
    *Q = int(sw / d->stride_w) + 1;
    // element counts must stay addressable with 63-bit offsets and per-dimension 31-bit indices
    const double big = 9e18;
    if (double(d->N) * d->H * d->W * d->C > big || double(d->N) * (*P) * (*Q) * d->K > big) return PCL_ERR_UNSUPPORTED_SHAPE;
    return PCL_OK;
}

bool unit_stride(const pcl_conv_desc& d) { return d.stride_h == 1 && d.stride_w == 1; }

// Which family a pass would use for this descriptor (pointer alignment is
// checked separately; all pointers are required to be 16-byte aligned anyway).
bool tensor_path_for(const pcl_conv_desc& d, int pass) {
    if (g_path.load() == PCL_PATH_GENERIC) return false;
    if (d.stride_h > 8 || d.stride_w > 8) return false;
    switch (pass) {
        case PCL_PASS_FWD: return d.C % 4 == 0;
        // (a strided layer runs one stride-1 sub-convolution per phase of the input grid, see conv_bwd_data_phases)
        case PCL_PASS_BWD_DATA: return d.K % 4 == 0 && (!unit_stride(d) || (d.pad_h <= d.R - 1 && d.pad_w <= d.S - 1));
        case PCL_PASS_BWD_WEIGHTS: return d.C % 4 == 0 && d.K % 4 == 0;
    }
    return false;
}

// Few-channel first layers (C < 4): the input is staged once as a 4-channel, halo-padded copy; a window of 8 pixels
// x 4 channels is then 32 contiguous floats, read through overlapping TMA windows (pixel stride 16 bytes, times the
// layer's stride).  The tensor-core kernels see a layer with 32 "channels" per tap, an R x S' kernel whose S' =
// ceil(S / 8) taps of a row lie 8 pixels apart (tap s' covers kernel columns 8s' .. 8s'+7; columns past S and the
// fourth channel meet zero weights), and no padding.
int few_sblocks(const pcl_conv_desc& d) { return (d.S + 7) / 8; }
bool few_channel_path_for(const pcl_conv_desc& d, int pass) {
    if (g_path.load() == PCL_PATH_GENERIC) return false;
    if (d.C >= 4 || d.S > 32 || d.stride_h > 8 || d.stride_w > 8) return false;
    if (pass == PCL_PASS_FWD) return true;
    if (pass == PCL_PASS_BWD_WEIGHTS) return d.K % 4 == 0;
    return false;
}
// The weight gradient of stride-1 few-channel layers with one window per kernel row and at most 8 rows takes all
// tap rows of a k tile in one work item (TcWgradArgs::tap_groups); other few-channel layers run the general form.
bool few_taprows_form(const pcl_conv_desc& d) { return unit_stride(d) && d.S <= 8 && d.R <= 8; }
int few_slack_pixels(const pcl_conv_desc& d) { return 8 * few_sblocks(d); }   // the last windows reach past the last row
size_t staged_x_bytes(const pcl_conv_desc& d) {
    return align_up((size_t(d.N) * (d.H + 2 * d.pad_h) * (d.W + 2 * d.pad_w) + few_slack_pixels(d)) * 16, 256);
}
size_t staged_w_bytes(const pcl_conv_desc& d) { return align_up(size_t(d.K) * d.R * few_sblocks(d) * 128, 256); }
// The staged layer as the forward-type kernel sees it.
TcFpropArgs few_fwd_args(const pcl_conv_desc& d, int P, int Q, const float* xs, const float* w4, const float* bias,
                         float* y, int act) {
    const int Hp = d.H + 2 * d.pad_h, Wp = d.W + 2 * d.pad_w, Sb = few_sblocks(d);
    // declared width: one window start per reachable pixel, (Q-1)*stride_w + 8*(S'-1) being the last
    TcFpropArgs a{xs, w4, bias, nullptr, y, d.N, Hp, (Q - 1) * d.stride_w + 8 * (Sb - 1) + 1, 32, d.K, d.R, Sb, 0, 0, P, Q, act};
    a.in_stride_w = 4; a.in_stride_h = long(Wp) * 4; a.in_stride_n = long(Hp) * Wp * 4;
    a.stride_h = d.stride_h; a.stride_w = d.stride_w; a.dil_w = Sb > 1 ? 8 : 1;     // (one window per row: no step between taps)
    a.k_live = Sb > 1 ? 0 : d.S * 4;      // one window per kernel row: only the first S*4 floats of it meet weights
    return a;
}

size_t dw_bytes(const pcl_conv_desc& d) { return align_up(size_t(d.K) * d.R * d.S * d.C * 4, 256); }

struct WgradPlan {
    bool few;            // few-channel staged path
    bool tensor;
    int splits;          // pixel splits of the main kernel
    size_t partial_bytes;
    size_t colsum_bytes;
};

WgradPlan plan_wgrad(const pcl_conv_desc& d, int P, int Q) {
    WgradPlan pl{};
    pl.few = few_channel_path_for(d, PCL_PASS_BWD_WEIGHTS);
    pl.tensor = pl.few || tensor_path_for(d, PCL_PASS_BWD_WEIGHTS);
    if (pl.few) {
        pl.splits = few_taprows_form(d) ? tc_wgrad_splits(d.N, P, Q, d.S * 4, d.K, d.R, 1, 1)
                                        : tc_wgrad_splits(d.N, P, Q, 32, d.K, d.R, few_sblocks(d), 0, 0, 1);
        // staged x + per-split dw4 tiles (always two-pass: the un-padding pass is needed anyway)
        pl.partial_bytes = staged_x_bytes(d) + size_t(pl.splits) * staged_w_bytes(d);
    } else {
        pl.splits = pl.tensor ? tc_wgrad_splits(d.N, P, Q, d.C, d.K, d.R, d.S, 0, 0, unit_stride(d) ? 0 : 1)
                              : generic_wgrad_splits(d, P, Q);
        pl.partial_bytes = pl.splits > 1 ? size_t(pl.splits) * dw_bytes(d) : 0;
    }
    const int cs = colsum_splits(size_t(d.N) * P * Q);
    pl.colsum_bytes = cs > 1 ? align_up(size_t(cs) * d.K * 4, 256) : 0;
    return pl;
}

// FC weight gradient dw[K][C] = dz^T[K][N] * x[N][C] through the forward-type kernel: its "pixels" are the K output
// rows, its reduction the minibatch, and x [N][C] is read in place as an MN-major weight operand; only dz has to be
// transposed (N*K floats).  The weight-gradient kernel proper is built for long reductions (one tile per CTA,
// epilogue not overlapped); with a minibatch-long reduction its tiles are mostly epilogue, while the forward-type
// kernel is persistent, overlaps a tile's epilogue with the next tile's MMAs and stores through TMA.
bool fc_dw_as_forward(int N, int C, int K) {
    if (g_path.load() == PCL_PATH_GENERIC) return false;
    if (N % 4 != 0 || C % 32 != 0 || K % 4 != 0) return false;
    if (tune_is_set(TUNE_FC_DW_FORWARD)) return tune(TUNE_FC_DW_FORWARD, 0) != 0;      // test / tuning hook
    // measured (B200): it pays for a short reduction and a large dw (VGG-A FC1: 0.26 -> 0.13 ms, FC2: 0.052 -> 0.039
    // with the transpose); at minibatch 1024 (the DNN layers) and for small dw the weight-gradient kernel is as fast
    return N <= 512 && size_t(K) * C >= (size_t(1) << 23);
}
size_t fc_dzt_bytes(int N, int K) { return align_up(size_t(N) * K * 4, 256); }

}  // namespace
}  // namespace pcl

using namespace pcl;

extern "C" {

int pcl_set_tuning(const char* name, int value) {
    if (!name) return PCL_ERR_BAD_ARG;
    for (int i = 0; i < TUNE_COUNT; ++i)
        if (strcmp(name, kTuneNames[i]) == 0) {
            g_tune[i].value.store(value);
            g_tune[i].set.store(value == INT_MIN ? 0 : 1);
            g_tune_gen.fetch_add(1);
            if (i == TUNE_WAIT_LIMIT_US) {       // lives in device memory next to the status word (current device)
                const unsigned int us = (value == INT_MIN || value <= 0) ? 2000000u : static_cast<unsigned int>(value);
                if (cudaMemcpyToSymbol(g_device_status, &us, sizeof(us), sizeof(unsigned int)) != cudaSuccess) return PCL_ERR_CUDA;
            }
            return PCL_OK;
        }
    return PCL_ERR_BAD_ARG;
}

int pcl_reset_tuning(void) {
    const bool had_limit = g_tune[TUNE_WAIT_LIMIT_US].set.load() != 0;
    for (int i = 0; i < TUNE_COUNT; ++i) g_tune[i].set.store(0);
    g_tune_gen.fetch_add(1);
    if (had_limit) {
        const unsigned int us = 2000000u;
        if (cudaMemcpyToSymbol(g_device_status, &us, sizeof(us), sizeof(unsigned int)) != cudaSuccess) return PCL_ERR_CUDA;
    }
    return PCL_OK;
}

int pcl_set_path(int path) {
    if (path != PCL_PATH_AUTO && path != PCL_PATH_TENSOR && path != PCL_PATH_GENERIC) return PCL_ERR_BAD_ARG;
    g_path.store(path);
    return PCL_OK;
}

int pcl_conv_out_dims(const pcl_conv_desc* d, int* P, int* Q) {
    if (!P || !Q) return PCL_ERR_BAD_ARG;
    return check_desc(d, P, Q);
}

// Scratch for a split reduction of the forward / backward-data launch (layers with few tiles and a long reduction:
// the FC layers at small minibatch); 0 where the launcher would not split.
static size_t fwd_split_bytes(const pcl_conv_desc& d, int P, int Q) {
    TcFpropArgs a{nullptr, nullptr, nullptr, nullptr, nullptr, d.N, d.H, d.W, d.C, d.K, d.R, d.S, d.pad_h, d.pad_w, P, Q,
                  PCL_ACT_NONE};
    a.stride_h = d.stride_h; a.stride_w = d.stride_w;
    return align_up(tc_fprop_split_ws_bytes(a), 256);
}
static size_t bwd_data_split_bytes(const pcl_conv_desc& d, int P, int Q) {
    if (d.stride_h != 1 || d.stride_w != 1) return 0;
    TcFpropArgs a{nullptr, nullptr, nullptr, nullptr, nullptr, d.N, P, Q, d.K, d.C, d.R, d.S,
                  d.R - 1 - d.pad_h, d.S - 1 - d.pad_w, d.H, d.W, PCL_ACT_NONE};
    if (d.C % 32 == 0) a.wt_mn_major = 1;       // (either form of the weights gives the same tiling)
    return align_up(tc_fprop_split_ws_bytes(a), 256);
}

size_t pcl_conv_workspace_bytes(const pcl_conv_desc* d, int pass) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    switch (pass) {
        case PCL_PASS_FWD:
            if (few_channel_path_for(*d, pass)) return staged_x_bytes(*d) + staged_w_bytes(*d);
            return tensor_path_for(*d, pass) ? fwd_split_bytes(*d, P, Q) : 0;
        case PCL_PASS_BWD_DATA:
            if (!tensor_path_for(*d, pass)) return 0;
            if (!unit_stride(*d)) return bwd_data_transposed_bytes(*d);
            return dw_bytes(*d) + bwd_data_split_bytes(*d, P, Q);
        case PCL_PASS_BWD_WEIGHTS: {
            const WgradPlan pl = plan_wgrad(*d, P, Q);
            return pl.partial_bytes + pl.colsum_bytes;
        }
    }
    return 0;
}

size_t pcl_fc_workspace_bytes(int N, int C, int K, int pass) {
    if (N <= 0 || C <= 0 || K <= 0) return 0;
    const pcl_conv_desc d{N, C, K, 1, 1, 1, 1, 1, 1, 0, 0};
    if (pass == PCL_PASS_FWD) return pcl_conv_workspace_bytes(&d, PCL_PASS_FWD);
    // fc_bwd runs both backward contractions; either pass value returns the total (the weight-gradient part is
    // sized for either of its two forms)
    const size_t wgrad_form = pcl_conv_workspace_bytes(&d, PCL_PASS_BWD_WEIGHTS);
    const size_t fwd_form = fc_dzt_bytes(N, K) + plan_wgrad(d, 1, 1).colsum_bytes;
    // (backward-data sized for its form with fused column sums, which contains the plain form)
    return pcl_conv_bwd_data_colsum_workspace_bytes(&d) + (wgrad_form > fwd_form ? wgrad_form : fwd_form);
}

// Forward pass; y_pool != nullptr: also the 2x2 window maxima of y, fused into the tensor-core epilogue where
// the shape allows it and computed by the pooling kernel otherwise.
static int conv_fwd_impl(const pcl_conv_desc* d, const float* x, const float* w, const float* bias, float* y,
                         float* y_pool, unsigned char* pool_codes, int act, void* ws, size_t ws_bytes,
                         void* cuda_stream) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!x || !w || (!y && !y_pool)) return PCL_ERR_BAD_ARG;
    PassScope pass_scope(PROF_PASS_CONV_FWD, conv_pass_flops(*d, P, Q));
    if (act != PCL_ACT_NONE && act != PCL_ACT_RELU && act != PCL_ACT_SIGMOID) return PCL_ERR_BAD_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(bias) || !aligned16(y_pool)) return PCL_ERR_MISALIGNED;
    // without y only the one-kernel form can run (the separate pooling kernel reads y)
    if (!y && !pcl_conv_fwd_pool_is_fused(d)) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (y_pool && (P % 2 != 0 || Q % 2 != 0)) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (pool_codes && (!y_pool || !aligned16(pool_codes))) return y_pool ? PCL_ERR_MISALIGNED : PCL_ERR_BAD_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (few_channel_path_for(*d, PCL_PASS_FWD)) {
        const size_t xs_bytes = staged_x_bytes(*d), need = xs_bytes + staged_w_bytes(*d);
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
        float* xs = static_cast<float*>(ws);
        float* w4 = reinterpret_cast<float*>(static_cast<char*>(ws) + xs_bytes);
        rc = launch_stage_pad_c4(x, xs, d->N, d->H, d->W, d->C, d->pad_h, d->pad_w, few_slack_pixels(*d), st);
        if (rc != PCL_OK) return rc;
        rc = launch_stage_w4(w, w4, size_t(d->K) * d->R, d->S, d->C, few_sblocks(*d) * 32, st);
        if (rc != PCL_OK) return rc;
        // the staged layer: 32 "channels" per pixel window (the taps' channels carry weight, the rest meets zero weights)
        TcFpropArgs a = few_fwd_args(*d, P, Q, xs, w4, bias, y, act);
        if (y_pool && tc_fprop_can_pool(a)) { a.pool_out = y_pool; a.pool_idx = pool_codes; y_pool = nullptr; }
        rc = launch_tc_fprop(a, st);
    } else if (tensor_path_for(*d, PCL_PASS_FWD)) {
        TcFpropArgs a{x, w, bias, nullptr, y, d->N, d->H, d->W, d->C, d->K, d->R, d->S, d->pad_h, d->pad_w, P, Q, act};
        a.stride_h = d->stride_h; a.stride_w = d->stride_w;
        if (y_pool && tc_fprop_can_pool(a)) { a.pool_out = y_pool; a.pool_idx = pool_codes; y_pool = nullptr; }
        if (ws && (reinterpret_cast<uintptr_t>(ws) & 255) == 0) {      // scratch for a split reduction, if the caller gave some
            a.split_ws = static_cast<float*>(ws); a.split_ws_bytes = ws_bytes;
        }
        rc = launch_tc_fprop(a, st);
    } else if (g_path.load() == PCL_PATH_TENSOR) {
        return PCL_ERR_UNSUPPORTED_SHAPE;
    } else {
        rc = launch_generic_fwd(*d, P, Q, x, w, bias, y, act, st);
    }
    if (rc != PCL_OK) return rc;
    if (y_pool) return launch_maxpool_fwd(d->N, P, Q, d->K, y, y_pool, st, pool_codes);     // not fused above
    return PCL_OK;
}

int pcl_conv_fwd_pool_is_fused(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    if (!few_channel_path_for(*d, PCL_PASS_FWD) && !tensor_path_for(*d, PCL_PASS_FWD)) return 0;
    TcFpropArgs a{};
    a.P = P; a.Q = Q; a.Kout = d->K;
    return tc_fprop_can_pool(a) ? 1 : 0;
}

int pcl_conv_fwd(const pcl_conv_desc* d, const float* x, const float* w, const float* bias, float* y, int act,
                 void* ws, size_t ws_bytes, void* cuda_stream) {
    return conv_fwd_impl(d, x, w, bias, y, nullptr, nullptr, act, ws, ws_bytes, cuda_stream);
}

int pcl_conv_fwd_pool(const pcl_conv_desc* d, const float* x, const float* w, const float* bias, float* y,
                      float* y_pool, unsigned char* pool_codes, int act, void* ws, size_t ws_bytes,
                      void* cuda_stream) {
    if (!y_pool) return PCL_ERR_BAD_ARG;
    return conv_fwd_impl(d, x, w, bias, y, y_pool, pool_codes, act, ws, ws_bytes, cuda_stream);
}

namespace {
// Backward-data of a strided layer on the tensor-core path.  Input pixel h belongs to phase a = (h + pad_h) mod
// stride_h (likewise b in w); only the taps r = a + i*stride_h reach it, from output rows p = (h + pad_h - a) /
// stride_h - i.  So every phase (a, b) is a stride-1 convolution of dy with the flipped sub-kernel
// w[k][a + i*stride_h][b + j*stride_w][c], written to every stride-th pixel of dx: stride_h * stride_w launches of
// the forward-type kernel, each with its own transposed sub-kernel in the workspace.  Pixels of phases without taps
// (a stride larger than the kernel) are zeroed first.
// Few input maps: all phases at once.  With h + pad_h = u*stride_h + a the rule reads
//   dx[n, h, w, c] = sum_{k, i, j} dy[n, u - i, v - j, k] * w[k, a + i*stride_h, b + j*stride_w, c],
// a stride-1 convolution of dy with a ceil(R/stride_h) x ceil(S/stride_w) kernel whose output map index is (a, b, c)
// (taps a phase does not have are zero weights); its output is scattered to dx by a bandwidth-bound pass.
int conv_bwd_data_packed(const pcl_conv_desc& d, const StridedBwdPlan& sp, int P, int Q, const float* dy, const float* w,
                         const float* mask, float* dx, char* ws, cudaStream_t st) {
    float* wpk = reinterpret_cast<float*>(ws);
    float* temp = reinterpret_cast<float*>(ws + sp.wpk_bytes);
    int rc = launch_phase_pack_weights(w, wpk, d.K, d.R, d.S, d.C, d.stride_h, d.stride_w, sp.Rm, sp.Sm, sp.cols4, st);
    if (rc != PCL_OK) return rc;
    TcFpropArgs t{dy, wpk, nullptr, nullptr, temp, d.N, P, Q, d.K, sp.cols4, sp.Rm, sp.Sm, sp.Rm - 1, sp.Sm - 1, sp.U, sp.V,
                  PCL_ACT_NONE};
    rc = launch_tc_fprop(t, st);
    if (rc != PCL_OK) return rc;
    return launch_phase_unpack(temp, mask, dx, d.N, d.H, d.W, d.C, d.stride_h, d.stride_w, d.pad_h, d.pad_w, sp.U, sp.V,
                               sp.cols4, st);
}

int conv_bwd_data_phases(const pcl_conv_desc& d, int P, int Q, const float* dy, const float* w, const float* mask,
                         float* dx, char* ws, cudaStream_t st) {
    const int sh = d.stride_h, sw = d.stride_w;
    if (sh > d.R || sw > d.S) {
        const int rc = launch_zero(dx, size_t(d.N) * d.H * d.W * d.C, st);
        if (rc != PCL_OK) return rc;
    }
    size_t off = 0;
    for (int a = 0; a < sh; ++a)
        for (int b = 0; b < sw; ++b) {
            const int Ra = a < d.R ? (d.R - a + sh - 1) / sh : 0, Sb = b < d.S ? (d.S - b + sw - 1) / sw : 0;
            if (Ra == 0 || Sb == 0) continue;
            // pixels of the phase: h + pad_h = u*stride_h + a with 0 <= h < H, i.e. u0 <= u <= u1
            const int u0 = d.pad_h > a ? (d.pad_h - a + sh - 1) / sh : 0, v0 = d.pad_w > b ? (d.pad_w - b + sw - 1) / sw : 0;
            const int top_h = d.H - 1 + d.pad_h - a, top_w = d.W - 1 + d.pad_w - b;
            if (top_h < 0 || top_w < 0) continue;
            const int Hph = top_h / sh - u0 + 1, Wph = top_w / sw - v0 + 1;
            if (Hph <= 0 || Wph <= 0) continue;
            float* wt = reinterpret_cast<float*>(ws + off);
            off += align_up(size_t(d.C) * Ra * Sb * d.K * 4, 256);
            int rc = launch_phase_weights(w, wt, d.K, d.R, d.S, d.C, a, b, sh, sw, Ra, Sb, st);
            if (rc != PCL_OK) return rc;
            const size_t first = (size_t(u0 * sh + a - d.pad_h) * d.W + size_t(v0 * sw + b - d.pad_w)) * d.C;
            // out[n, u', v', c] = sum_{r', s', k} dy[n, u' + r' - (Ra-1-u0), v' + s' - (Sb-1-v0), k] * wt[c][r'][s'][k]
            TcFpropArgs t{dy, wt, nullptr, mask ? mask + first : nullptr, dx + first, d.N, P, Q, d.K, d.C, Ra, Sb,
                          Ra - 1 - u0, Sb - 1 - v0, Hph, Wph, PCL_ACT_NONE};
            t.out_stride_w = long(sw) * d.C; t.out_stride_h = long(sh) * d.W * d.C; t.out_stride_n = long(d.H) * d.W * d.C;
            rc = launch_tc_fprop(t, st);
            if (rc != PCL_OK) return rc;
        }
    return PCL_OK;
}
}  // namespace

int pcl_conv_bwd_data(const pcl_conv_desc* d, const float* dy, const float* w, const float* relu_mask_src, float* dx,
                      void* ws, size_t ws_bytes, void* cuda_stream) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!dy || !w || !dx) return PCL_ERR_BAD_ARG;
    PassScope pass_scope(PROF_PASS_CONV_BWD_DATA, conv_pass_flops(*d, P, Q));
    if (!aligned16(dy) || !aligned16(w) || !aligned16(dx) || !aligned16(relu_mask_src)) return PCL_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (tensor_path_for(*d, PCL_PASS_BWD_DATA)) {
        // mandatory: room for the transposed copy where one is made; whatever follows it is optional scratch for
        // a split reduction (the launcher splits as far as that room allows, or not at all)
        const size_t need = bwd_data_transposed_bytes(*d);
        if (need > 0 && (!ws || ws_bytes < need)) return PCL_ERR_WORKSPACE;
        if (ws && (reinterpret_cast<uintptr_t>(ws) & 255)) return PCL_ERR_MISALIGNED;
        if (!unit_stride(*d)) {
            const StridedBwdPlan sp = strided_bwd_plan(*d);
            if (sp.packed && tune(TUNE_PACKED_BWD, 1))
                return conv_bwd_data_packed(*d, sp, P, Q, dy, w, relu_mask_src, dx, static_cast<char*>(ws), st);
            if (ws_bytes < dw_bytes(*d) + size_t(256) * d->stride_h * d->stride_w) return PCL_ERR_WORKSPACE;
            return conv_bwd_data_phases(*d, P, Q, dy, w, relu_mask_src, dx, static_cast<char*>(ws), st);
        }
        // dx = "forward" convolution of dy with the flipped, transposed weights, pad' = R-1-pad
        TcFpropArgs a{dy, w, nullptr, relu_mask_src, dx, d->N, P, Q, d->K, d->C, d->R, d->S,
                      d->R - 1 - d->pad_h, d->S - 1 - d->pad_w, d->H, d->W, PCL_ACT_NONE};
        if (ws && ws_bytes > need) {
            a.split_ws = reinterpret_cast<float*>(static_cast<char*>(ws) + need); a.split_ws_bytes = ws_bytes - need;
        }
        if (weights_read_in_place(*d)) {
            // the kernel reads w itself as an MN-major operand (taps flipped by index): no transposed copy
            a.wt_mn_major = 1; a.flip_taps = 1;
        } else {
            float* wt_t = static_cast<float*>(ws);
            rc = launch_transpose_flip(w, wt_t, d->K, d->R, d->S, d->C, st);
            if (rc != PCL_OK) return rc;
            a.wt = wt_t;
        }
        return launch_tc_fprop(a, st);
    }
    if (g_path.load() == PCL_PATH_TENSOR) return PCL_ERR_UNSUPPORTED_SHAPE;
    return launch_generic_bwd_data(*d, P, Q, dy, w, relu_mask_src, dx, st);
}

namespace {
// Workspace layout of the fused "dx + column sums of dx" calls: [main pass scratch][per-tile / per-block sum rows]
// [second-stage partials of the column sum over those rows].
size_t colsum_stage_bytes(long rows, int cols) {
    if (rows <= 0) return 0;
    const int cs = colsum_splits(size_t(rows));
    return align_up(size_t(rows) * cols * 4, 256) + (cs > 1 ? align_up(size_t(cs) * cols * 4, 256) : 0);
}
// `w` is the layer's own KRSC tensor when the kernel can read it in place, else the caller puts the transposed copy in.
TcFpropArgs bwd_data_args(const pcl_conv_desc& d, int P, int Q, const float* dy, const float* w,
                          const float* mask, float* dx) {
    TcFpropArgs a{dy, w, nullptr, mask, dx, d.N, P, Q, d.K, d.C, d.R, d.S,
                  d.R - 1 - d.pad_h, d.S - 1 - d.pad_w, d.H, d.W, PCL_ACT_NONE};
    if (weights_read_in_place(d)) { a.wt_mn_major = 1; a.flip_taps = 1; }
    return a;
}
}  // namespace

int pcl_conv_plan_describe(const pcl_conv_desc* d, int pass, char* buf, size_t buf_bytes) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!buf || buf_bytes < 64) return PCL_ERR_BAD_ARG;
    const float* fake = reinterpret_cast<const float*>(uintptr_t(256));      // (alignment checks only; nothing is read)
    if (pass == PCL_PASS_FWD && few_channel_path_for(*d, pass)) {
        return tc_fprop_describe(few_fwd_args(*d, P, Q, fake, fake, nullptr, const_cast<float*>(fake), PCL_ACT_RELU), buf, buf_bytes);
    } else if (pass == PCL_PASS_FWD && tensor_path_for(*d, pass)) {
        TcFpropArgs a{fake, fake, nullptr, nullptr, const_cast<float*>(fake), d->N, d->H, d->W, d->C, d->K, d->R, d->S,
                      d->pad_h, d->pad_w, P, Q, PCL_ACT_RELU};
        a.stride_h = d->stride_h; a.stride_w = d->stride_w;
        return tc_fprop_describe(a, buf, buf_bytes);
    } else if (pass == PCL_PASS_BWD_DATA && tensor_path_for(*d, pass) && unit_stride(*d)) {
        return tc_fprop_describe(bwd_data_args(*d, P, Q, fake, fake, nullptr, const_cast<float*>(fake)), buf, buf_bytes);
    }
    snprintf(buf, buf_bytes, "not a single forward-type tensor-core launch");
    return PCL_OK;
}

size_t pcl_conv_bwd_data_colsum_workspace_bytes(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    const size_t base = pcl_conv_workspace_bytes(d, PCL_PASS_BWD_DATA);
    long rows = 0;
    if (tensor_path_for(*d, PCL_PASS_BWD_DATA) && d->C % 4 == 0 && unit_stride(*d))
        rows = tc_fprop_colsum_rows(bwd_data_args(*d, P, Q, nullptr, nullptr, nullptr, nullptr));
    if (rows > 0) return base + colsum_stage_bytes(rows, d->C);
    const int cs = colsum_splits(size_t(d->N) * d->H * d->W);          // unfused: column sum of dx itself
    return base + (cs > 1 ? align_up(size_t(cs) * d->C * 4, 256) : 0);
}

namespace {
// Backward-data with the gradient of the activation that produced `mask` folded into the epilogue (mask_mode 0: ReLU,
// 1: sigmoid) and, if dx_colsum != nullptr, the per-map sums of what was written.  Workspace layout as
// pcl_conv_bwd_data_colsum_workspace_bytes() describes.
int bwd_data_masked_colsum(const pcl_conv_desc* d, int P, int Q, const float* dy, const float* w, const float* mask,
                           int mask_mode, float* dx, float* dx_colsum, void* ws, size_t ws_bytes, void* cuda_stream) {
    const size_t need = dx_colsum ? pcl_conv_bwd_data_colsum_workspace_bytes(d) : bwd_data_transposed_bytes(*d);
    if (need > 0) {
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t base = pcl_conv_workspace_bytes(d, PCL_PASS_BWD_DATA);
    const bool tensor = tensor_path_for(*d, PCL_PASS_BWD_DATA) && unit_stride(*d);
    int rc;
    if (tensor) {
        long rows = 0;
        if (dx_colsum && d->C % 4 == 0) rows = tc_fprop_colsum_rows(bwd_data_args(*d, P, Q, nullptr, nullptr, nullptr, nullptr));
        TcFpropArgs a = bwd_data_args(*d, P, Q, dy, w, mask, dx);
        a.mask_mode = mask_mode;
        if (!a.wt_mn_major) {
            float* wt_t = static_cast<float*>(ws);
            rc = launch_transpose_flip(w, wt_t, d->K, d->R, d->S, d->C, st);
            if (rc != PCL_OK) return rc;
            a.wt = wt_t;
        }
        if (rows > 0) {
            char* extra = static_cast<char*>(ws) + base;
            float* sum_rows = reinterpret_cast<float*>(extra);
            a.colsum_rows = sum_rows;
            // (the workspace is sized for the tiling with the most rows; this launch writes rows 0 .. written-1, of which a
            // grid smaller than the device leaves some untouched: those must not contribute)
            bool all_written = false;
            long written = tc_fprop_colsum_rows_written(a, &all_written);
            if (written <= 0 || written > rows) { written = rows; all_written = false; }
            if (!all_written) {
                rc = launch_zero(sum_rows, size_t(written) * d->C, st);
                if (rc != PCL_OK) return rc;
            }
            rc = launch_tc_fprop(a, st);
            if (rc != PCL_OK) return rc;
            float* partial = reinterpret_cast<float*>(extra + align_up(size_t(rows) * d->C * 4, 256));
            return launch_colsum(sum_rows, size_t(written), d->C, partial, dx_colsum, st);
        }
        if (!dx_colsum && !mask && ws && ws_bytes > bwd_data_transposed_bytes(*d)) {      // room to split a long reduction
            const size_t t = bwd_data_transposed_bytes(*d);
            a.split_ws = reinterpret_cast<float*>(static_cast<char*>(ws) + t); a.split_ws_bytes = ws_bytes - t;
        }
        rc = launch_tc_fprop(a, st);
        if (rc != PCL_OK) return rc;
    } else {
        // other kernel families: backward-data with the ReLU mask they know, any other gradient as a pass over dx
        rc = pcl_conv_bwd_data(d, dy, w, mask_mode == 0 ? mask : nullptr, dx, ws, base, cuda_stream);
        if (rc != PCL_OK) return rc;
        if (mask && mask_mode == 1) {
            rc = launch_act_grad(dx, mask, size_t(d->N) * d->H * d->W * d->C, PCL_ACT_SIGMOID, st);
            if (rc != PCL_OK) return rc;
        }
    }
    if (!dx_colsum) return PCL_OK;
    char* extra = static_cast<char*>(ws) + base;
    return launch_colsum(dx, size_t(d->N) * d->H * d->W, d->C, reinterpret_cast<float*>(extra), dx_colsum, st);
}
}  // namespace

int pcl_conv_bwd_data_colsum(const pcl_conv_desc* d, const float* dy, const float* w, const float* relu_mask_src,
                             float* dx, float* dx_colsum, void* ws, size_t ws_bytes, void* cuda_stream) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!dy || !w || !dx || !dx_colsum) return PCL_ERR_BAD_ARG;
    PassScope pass_scope(PROF_PASS_CONV_BWD_DATA, conv_pass_flops(*d, P, Q));
    if (!aligned16(dy) || !aligned16(w) || !aligned16(dx) || !aligned16(relu_mask_src) || !aligned16(dx_colsum))
        return PCL_ERR_MISALIGNED;
    return bwd_data_masked_colsum(d, P, Q, dy, w, relu_mask_src, 0, dx, dx_colsum, ws, ws_bytes, cuda_stream);
}

size_t pcl_maxpool2x2_bwd_colsum_workspace_bytes(int N, int H, int W, int C) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0) return 0;
    const long rows = maxpool_bwd_colsum_rows(N, H, W, C);
    if (rows > 0) return colsum_stage_bytes(rows, C);
    const int cs = colsum_splits(size_t(N) * H * W);
    return cs > 1 ? align_up(size_t(cs) * C * 4, 256) : 0;
}

int pcl_maxpool2x2_bwd_colsum(int N, int H, int W, int C, const float* x, const float* dy, const float* relu_mask_src,
                              float* dx, float* dx_colsum, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !x || !dy || !dx || !dx_colsum) return PCL_ERR_BAD_ARG;
    if ((H | W) & 1) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(relu_mask_src) || !aligned16(dx_colsum))
        return PCL_ERR_MISALIGNED;
    const size_t need = pcl_maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C);
    if (need > 0) {
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const long rows = maxpool_bwd_colsum_rows(N, H, W, C);
    if (rows > 0) {
        float* sum_rows = static_cast<float*>(ws);
        int rc = launch_maxpool_bwd_colsum(N, H, W, C, x, dy, relu_mask_src, dx, sum_rows, st);
        if (rc != PCL_OK) return rc;
        float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) + align_up(size_t(rows) * C * 4, 256));
        return launch_colsum(sum_rows, size_t(rows), C, partial, dx_colsum, st);
    }
    int rc = launch_maxpool_bwd(N, H, W, C, x, dy, relu_mask_src, dx, st);
    if (rc != PCL_OK) return rc;
    return launch_colsum(dx, size_t(N) * H * W, C, static_cast<float*>(ws), dx_colsum, st);
}

int pcl_maxpool2x2_fwd_codes(int N, int H, int W, int C, const float* x, float* y, unsigned char* codes,
                             void* cuda_stream) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !x || !y || !codes) return PCL_ERR_BAD_ARG;
    if ((H | W) & 1) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(x) || !aligned16(y) || !aligned16(codes)) return PCL_ERR_MISALIGNED;
    return launch_maxpool_fwd(N, H, W, C, x, y, static_cast<cudaStream_t>(cuda_stream), codes);
}

int pcl_maxpool2x2_bwd_codes(int N, int H, int W, int C, const unsigned char* codes, const float* dy, int relu_mask,
                             float* dx, float* dx_colsum, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !codes || !dy || !dx) return PCL_ERR_BAD_ARG;
    if ((H | W) & 1) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(codes) || !aligned16(dy) || !aligned16(dx) || !aligned16(dx_colsum)) return PCL_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!dx_colsum) return launch_maxpool_bwd_idx(N, H, W, C, codes, dy, relu_mask, dx, nullptr, st);
    const size_t need = pcl_maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C);
    if (need > 0) {
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    const long rows = maxpool_bwd_colsum_rows(N, H, W, C);
    if (rows > 0) {
        float* sum_rows = static_cast<float*>(ws);
        int rc = launch_maxpool_bwd_idx(N, H, W, C, codes, dy, relu_mask, dx, sum_rows, st);
        if (rc != PCL_OK) return rc;
        float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) + align_up(size_t(rows) * C * 4, 256));
        return launch_colsum(sum_rows, size_t(rows), C, partial, dx_colsum, st);
    }
    int rc = launch_maxpool_bwd_idx(N, H, W, C, codes, dy, relu_mask, dx, nullptr, st);
    if (rc != PCL_OK) return rc;
    return launch_colsum(dx, size_t(N) * H * W, C, static_cast<float*>(ws), dx_colsum, st);
}

namespace {
// Pooled-dy form of the few-channel weight gradient: splits and workspace layout [staged x][per-split dw tiles]
// [per-split bias-gradient rows].
struct PooledWgradPlan { bool ok; int splits; size_t tiles_off, rows_off, cs_off, total; };
PooledWgradPlan plan_pooled_wgrad(const pcl_conv_desc& d, int P, int Q) {
    PooledWgradPlan pl{};
    if (!few_channel_path_for(d, PCL_PASS_BWD_WEIGHTS) || !few_taprows_form(d)) return pl;
    if (!tc_wgrad_can_take_pooled_dy(d.N, P, Q, d.S * 4, d.K, d.R, 1, 1)) return pl;
    pl.ok = true;
    pl.splits = tc_wgrad_splits(d.N, P, Q, d.S * 4, d.K, d.R, 1, 1, 1);
    pl.tiles_off = staged_x_bytes(d);
    pl.rows_off = pl.tiles_off + size_t(pl.splits) * staged_w_bytes(d);
    pl.cs_off = pl.rows_off + align_up(size_t(pl.splits) * kPooledDbRows * d.K * 4, 256);      // one row per (split, builder warp)
    const int cs = colsum_splits(size_t(pl.splits) * kPooledDbRows);
    pl.total = pl.cs_off + (cs > 1 ? align_up(size_t(cs) * d.K * 4, 256) : 0);
    return pl;
}
}  // namespace

int pcl_conv_bwd_weights_pooled_is_fused(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    return plan_pooled_wgrad(*d, P, Q).ok ? 1 : 0;
}

size_t pcl_conv_bwd_weights_pooled_workspace_bytes(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    return plan_pooled_wgrad(*d, P, Q).total;
}

size_t pcl_conv_staged_input_bytes(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    return few_channel_path_for(*d, PCL_PASS_FWD) ? staged_x_bytes(*d) : 0;
}

static int conv_bwd_weights_pooled_impl(const pcl_conv_desc* d, const float* x, const float* x_staged, const float* dy_pool,
                                        const unsigned char* pool_codes, int relu_mask, float* dw, float* dbias, void* ws,
                                        size_t ws_bytes, void* cuda_stream) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if ((!x && !x_staged) || !dy_pool || !pool_codes || !dw) return PCL_ERR_BAD_ARG;
    if (x_staged && (reinterpret_cast<uintptr_t>(x_staged) & 255)) return PCL_ERR_MISALIGNED;
    PassScope pass_scope(PROF_PASS_CONV_BWD_WEIGHTS, conv_pass_flops(*d, P, Q));
    if (!aligned16(x) || !aligned16(dy_pool) || !aligned16(pool_codes) || !aligned16(dw) || !aligned16(dbias))
        return PCL_ERR_MISALIGNED;
    const PooledWgradPlan pl = plan_pooled_wgrad(*d, P, Q);
    if (!pl.ok) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!ws || ws_bytes < pl.total) return PCL_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the staged copy: the caller's (left by this layer's forward call at the start of its workspace), or made here
    const float* xs = x_staged ? x_staged : static_cast<const float*>(ws);
    float* dw4 = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.tiles_off);
    float* rows = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.rows_off);
    float* cs = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.cs_off);
    if (!x_staged) {
        rc = launch_stage_pad_c4(x, static_cast<float*>(ws), d->N, d->H, d->W, d->C, d->pad_h, d->pad_w, few_slack_pixels(*d), st);
        if (rc != PCL_OK) return rc;
    }
    const int Hp = d->H + 2 * d->pad_h, Wp = d->W + 2 * d->pad_w;
    const size_t taps = size_t(d->K) * d->R * d->S;
    TcWgradArgs a{xs, nullptr, dw4, pl.splits > 1 ? dw4 : nullptr, d->N, Hp, Q, d->S * 4, d->K, d->R, 1, 0, 0, P, Q,
                  pl.splits};
    a.x_stride_w = 4; a.x_stride_h = long(Wp) * 4; a.x_stride_n = long(Hp) * Wp * 4;
    a.x_inner = 32;
    a.tap_groups = 1;
    a.skip_reduce = 1;
    a.dy_pool = dy_pool; a.codes = pool_codes; a.relu_mask = relu_mask ? 1 : 0; a.db_rows = dbias ? rows : nullptr;
    rc = launch_tc_wgrad(a, st);
    if (rc != PCL_OK) return rc;
    rc = launch_unpad_reduce(dw4, dw, size_t(d->K) * d->R, d->S, d->C, d->S * 4, pl.splits, taps * 4, st);
    if (rc != PCL_OK) return rc;
    if (dbias) rc = launch_colsum(rows, size_t(pl.splits) * kPooledDbRows, d->K, cs, dbias, st);       // adds the rows, fixed order
    return rc;
}

int pcl_conv_bwd_weights_pooled(const pcl_conv_desc* d, const float* x, const float* dy_pool,
                                const unsigned char* pool_codes, int relu_mask, float* dw, float* dbias, void* ws,
                                size_t ws_bytes, void* cuda_stream) {
    if (!x) return PCL_ERR_BAD_ARG;
    return conv_bwd_weights_pooled_impl(d, x, nullptr, dy_pool, pool_codes, relu_mask, dw, dbias, ws, ws_bytes, cuda_stream);
}

int pcl_conv_bwd_weights_pooled_staged(const pcl_conv_desc* d, const float* x_staged, const float* dy_pool,
                                       const unsigned char* pool_codes, int relu_mask, float* dw, float* dbias, void* ws,
                                       size_t ws_bytes, void* cuda_stream) {
    if (!x_staged) return PCL_ERR_BAD_ARG;
    return conv_bwd_weights_pooled_impl(d, nullptr, x_staged, dy_pool, pool_codes, relu_mask, dw, dbias, ws, ws_bytes, cuda_stream);
}

namespace {
// Workspace of the fused-update form behind the plain form's: a dw-sized scratch, unless the update rides on the second
// pass of a split reduction (tensor path, more than one pixel split), which never forms dw.
bool sgd_rides_on_reduction(const pcl_conv_desc& d, int P, int Q) {
    const WgradPlan pl = plan_wgrad(d, P, Q);
    return pl.tensor && !pl.few;      // (more than one pixel split: the second pass; one: the kernel's epilogue)
}
int conv_bwd_weights_impl(const pcl_conv_desc* d, const float* x, const float* dy, float* dw, float* dbias, int deterministic,
                          void* ws, size_t ws_bytes, void* cuda_stream, float* w_update, float lr);
}  // namespace

int pcl_conv_bwd_weights(const pcl_conv_desc* d, const float* x, const float* dy, float* dw, float* dbias,
                         int deterministic, void* ws, size_t ws_bytes, void* cuda_stream) {
    return conv_bwd_weights_impl(d, x, dy, dw, dbias, deterministic, ws, ws_bytes, cuda_stream, nullptr, 0.f);
}

size_t pcl_conv_bwd_weights_sgd_workspace_bytes(const pcl_conv_desc* d) {
    int P, Q;
    if (check_desc(d, &P, &Q) != PCL_OK) return 0;
    const size_t base = align_up(pcl_conv_workspace_bytes(d, PCL_PASS_BWD_WEIGHTS), 256);
    return sgd_rides_on_reduction(*d, P, Q) ? base : base + align_up(dw_bytes(*d), 256);
}

int pcl_conv_bwd_weights_sgd(const pcl_conv_desc* d, const float* x, const float* dy, float* w, float lr, float* dbias,
                             void* ws, size_t ws_bytes, void* cuda_stream) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!w) return PCL_ERR_BAD_ARG;
    if (!aligned16(w)) return PCL_ERR_MISALIGNED;
    const size_t need = pcl_conv_bwd_weights_sgd_workspace_bytes(d);
    if (need > 0) {
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    if (sgd_rides_on_reduction(*d, P, Q))
        return conv_bwd_weights_impl(d, x, dy, w /* unused as dw */, dbias, 1, ws, ws_bytes, cuda_stream, w, lr);
    // no split reduction to ride on: dw goes to the scratch behind the plain form's workspace, then the update
    const size_t base = align_up(pcl_conv_workspace_bytes(d, PCL_PASS_BWD_WEIGHTS), 256);
    float* dw = reinterpret_cast<float*>(static_cast<char*>(ws) + base);
    rc = conv_bwd_weights_impl(d, x, dy, dw, dbias, 1, ws, base, cuda_stream, nullptr, 0.f);
    if (rc != PCL_OK) return rc;
    return launch_sgd(w, dw, size_t(d->K) * d->R * d->S * d->C, lr, static_cast<cudaStream_t>(cuda_stream));
}

namespace {
int conv_bwd_weights_impl(const pcl_conv_desc* d, const float* x, const float* dy, float* dw, float* dbias, int deterministic,
                          void* ws, size_t ws_bytes, void* cuda_stream, float* w_update, float lr) {
    int P, Q;
    int rc = check_desc(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    if (!x || !dy || !dw) return PCL_ERR_BAD_ARG;
    PassScope pass_scope(PROF_PASS_CONV_BWD_WEIGHTS, conv_pass_flops(*d, P, Q));
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dw) || !aligned16(dbias)) return PCL_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const WgradPlan pl = plan_wgrad(*d, P, Q);
    if (!pl.tensor && g_path.load() == PCL_PATH_TENSOR) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (pl.few) {
        const size_t xs_bytes = staged_x_bytes(*d);
        const size_t need_few = pl.partial_bytes + (dbias ? pl.colsum_bytes : 0);
        if (!ws || ws_bytes < need_few) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
        float* xs = static_cast<float*>(ws);
        float* dw4 = reinterpret_cast<float*>(static_cast<char*>(ws) + xs_bytes);
        float* cs = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.partial_bytes);
        rc = launch_stage_pad_c4(x, xs, d->N, d->H, d->W, d->C, d->pad_h, d->pad_w, few_slack_pixels(*d), st);
        if (rc != PCL_OK) return rc;
        const int Hp = d->H + 2 * d->pad_h, Wp = d->W + 2 * d->pad_w;
        const size_t taps = size_t(d->K) * d->R * d->S;
        if (few_taprows_form(*d)) {
            // partial tiles always go to the workspace (splits == 1 included): dw4 is [split][K][R][S*4]
            TcWgradArgs a{xs, dy, dw4, pl.splits > 1 ? dw4 : nullptr, d->N, Hp, Q, d->S * 4, d->K, d->R, 1, 0, 0, P, Q,
                          pl.splits};
            a.x_stride_w = 4; a.x_stride_h = long(Wp) * 4; a.x_stride_n = long(Hp) * Wp * 4;
            a.x_inner = 32;
            a.tap_groups = 1;
            a.skip_reduce = 1;
            rc = launch_tc_wgrad(a, st);
            if (rc != PCL_OK) return rc;
            rc = launch_unpad_reduce(dw4, dw, size_t(d->K) * d->R, d->S, d->C, d->S * 4, pl.splits, taps * 4, st);
        } else {
            // general form: a layer with 32 "channels" per tap and an R x S' kernel whose taps lie 8 pixels apart;
            // dw4 is [split][K][R][S'][32]
            const int Sb = few_sblocks(*d);
            const size_t tile = size_t(d->K) * d->R * Sb * 32;
            TcWgradArgs a{xs, dy, dw4, pl.splits > 1 ? dw4 : nullptr, d->N, Hp, (Q - 1) * d->stride_w + 8 * (Sb - 1) + 1, 32,
                          d->K, d->R, Sb, 0, 0, P, Q, pl.splits};
            a.x_stride_w = 4; a.x_stride_h = long(Wp) * 4; a.x_stride_n = long(Hp) * Wp * 4;
            a.x_inner = 32;
            a.stride_h = d->stride_h; a.stride_w = d->stride_w; a.dil_w = Sb > 1 ? 8 : 1;
            a.skip_reduce = 1;
            rc = launch_tc_wgrad(a, st);
            if (rc != PCL_OK) return rc;
            rc = launch_unpad_reduce(dw4, dw, size_t(d->K) * d->R, d->S, d->C, Sb * 32, pl.splits, tile, st);
        }
        if (rc != PCL_OK) return rc;
        if (dbias) rc = launch_colsum(dy, size_t(d->N) * P * Q, d->K, cs, dbias, st);
        return rc;
    }
    const bool need_partial = pl.splits > 1 && (deterministic || !pl.tensor);
    size_t need = (need_partial ? pl.partial_bytes : 0) + (dbias ? pl.colsum_bytes : 0);
    if (need > 0) {
        if (!ws || ws_bytes < need) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    float* partial = need_partial ? static_cast<float*>(ws) : nullptr;
    float* cs_partial = reinterpret_cast<float*>(static_cast<char*>(ws) + (need_partial ? pl.partial_bytes : 0));
    if (pl.tensor) {
        TcWgradArgs a{x, dy, dw, partial, d->N, d->H, d->W, d->C, d->K, d->R, d->S, d->pad_h, d->pad_w, P, Q, pl.splits};
        a.stride_h = d->stride_h; a.stride_w = d->stride_w;
        if (w_update && pl.splits > 1) {      // the second pass of the split reduction applies the update
            if (!partial) return PCL_ERR_BAD_ARG;
            a.skip_reduce = 1;
        } else if (w_update) {                // unsplit: the kernel's epilogue does
            a.w_update = w_update; a.lr = lr;
        }
        rc = launch_tc_wgrad(a, st);
        if (rc == PCL_OK && w_update && pl.splits > 1)
            rc = launch_reduce_splits_sgd(partial, w_update, size_t(d->K) * d->R * d->S * d->C, pl.splits, lr, st);
    } else {
        if (w_update) return PCL_ERR_BAD_ARG;
        rc = launch_generic_bwd_weights(*d, P, Q, x, dy, dw, partial, pl.splits, st);
    }
    if (rc != PCL_OK) return rc;
    if (dbias) rc = launch_colsum(dy, size_t(d->N) * P * Q, d->K, cs_partial, dbias, st);
    return rc;
}
}  // namespace

int pcl_fc_fwd(int N, int C, int K, const float* x, const float* w, const float* bias, float* y, int act, void* ws,
               size_t ws_bytes, void* cuda_stream) {
    const pcl_conv_desc d{N, C, K, 1, 1, 1, 1, 1, 1, 0, 0};
    PassScope pass_scope(PROF_PASS_FC_FWD, 2.0 * N * double(C) * K);
    return pcl_conv_fwd(&d, x, w, bias, y, act, ws, ws_bytes, cuda_stream);
}

namespace {
bool known_act(int act) { return act == PCL_ACT_NONE || act == PCL_ACT_RELU || act == PCL_ACT_SIGMOID; }

// w_update (with lr): the layer's weights are updated in place, w <- w - lr * dw, and dw is not stored (`dw` is ignored);
// backpropagation, which reads the old weights, then runs first.
int fc_bwd_impl(int N, int C, int K, const float* x, const float* w, const float* y, int act, float* dy, float* dx,
                int x_act, float* dx_colsum, float* dw, float* dbias, void* ws, size_t ws_bytes, void* cuda_stream,
                float* w_update = nullptr, float lr = 0.f) {
    if (N <= 0 || C <= 0 || K <= 0) return PCL_ERR_BAD_ARG;
    if (w_update) dw = w_update;      // (only its alignment is looked at below)
    if (!x || !w || !dy || !dw) return PCL_ERR_BAD_ARG;
    if (!known_act(act) || !known_act(x_act)) return PCL_ERR_BAD_ARG;
    if (act != PCL_ACT_NONE && !y) return PCL_ERR_BAD_ARG;
    if (!dx && dx_colsum) return PCL_ERR_BAD_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(dy) || !aligned16(dx) || !aligned16(dw) ||
        !aligned16(dbias) || !aligned16(dx_colsum))
        return PCL_ERR_MISALIGNED;
    const pcl_conv_desc d{N, C, K, 1, 1, 1, 1, 1, 1, 0, 0};
    const bool dw_fwd = fc_dw_as_forward(N, C, K);
    PassScope pass_scope(PROF_PASS_FC_BWD, 2.0 * N * double(C) * K, dx ? 2 : 1);
    const size_t colsum_bytes = plan_wgrad(d, 1, 1).colsum_bytes;
    const size_t need_w = dw_fwd ? fc_dzt_bytes(N, K) + colsum_bytes
                                 : (w_update ? pcl_conv_bwd_weights_sgd_workspace_bytes(&d)
                                             : pcl_conv_workspace_bytes(&d, PCL_PASS_BWD_WEIGHTS));
    const bool fused_dx = dx && (x_act != PCL_ACT_NONE || dx_colsum);
    const size_t need_d = !dx ? 0 : (dx_colsum ? pcl_conv_bwd_data_colsum_workspace_bytes(&d)
                                               : pcl_conv_workspace_bytes(&d, PCL_PASS_BWD_DATA));
    if (need_w + need_d > 0) {
        if (!ws || ws_bytes < need_w + need_d) return PCL_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(ws) & 255) return PCL_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int rc = launch_act_grad(dy, y, size_t(N) * K, act, st);
    if (rc != PCL_OK) return rc;
    char* ws_d = static_cast<char*>(ws) + need_w;
    auto backprop = [&]() -> int {
        if (!dx) return PCL_OK;
        if (!fused_dx) return pcl_conv_bwd_data(&d, dy, w, nullptr, dx, ws_d, need_d, cuda_stream);
        // dx = (dz w) times the gradient of the activation that produced x: what the layer below needs as its dz
        return bwd_data_masked_colsum(&d, 1, 1, dy, w, x_act == PCL_ACT_NONE ? nullptr : x, x_act == PCL_ACT_SIGMOID ? 1 : 0, dx,
                                      dx_colsum, ws_d, need_d, cuda_stream);
    };
    if (w_update) {       // in-place update: the old weights are read first
        rc = backprop();
        if (rc != PCL_OK) return rc;
    }
    // weight gradient first, then backpropagation (the order Sec. 3.1 schedules them in)
    if (dw_fwd) {
        float* dzt = static_cast<float*>(ws);
        float* cs = reinterpret_cast<float*>(static_cast<char*>(ws) + fc_dzt_bytes(N, K));
        rc = launch_transpose_flip(dy, dzt, N, 1, 1, K, st);       // dzt[k][n] = dz[n][k]
        if (rc != PCL_OK) return rc;
        TcFpropArgs a{dzt, x, nullptr, nullptr, dw, K, 1, 1, N, C, 1, 1, 0, 0, 1, 1, PCL_ACT_NONE};
        a.wt_mn_major = 1;
        if (w_update) { a.mask_src = w_update; a.mask_mode = 2; a.lr = lr; a.out = w_update; }     // w - lr * dw, in place
        rc = launch_tc_fprop(a, st);
        if (rc == PCL_OK && dbias) rc = launch_colsum(dy, size_t(N), K, cs, dbias, st);
    } else if (w_update) {
        rc = pcl_conv_bwd_weights_sgd(&d, x, dy, w_update, lr, dbias, ws, need_w, cuda_stream);
    } else {
        rc = pcl_conv_bwd_weights(&d, x, dy, dw, dbias, 1, ws, need_w, cuda_stream);
    }
    if (rc != PCL_OK) return rc;
    return w_update ? PCL_OK : backprop();
}
}  // namespace

int pcl_fc_bwd(int N, int C, int K, const float* x, const float* w, const float* y, int act, float* dy, float* dx,
               float* dw, float* dbias, void* ws, size_t ws_bytes, void* cuda_stream) {
    return fc_bwd_impl(N, C, K, x, w, y, act, dy, dx, PCL_ACT_NONE, nullptr, dw, dbias, ws, ws_bytes, cuda_stream);
}

int pcl_fc_bwd_fused(int N, int C, int K, const float* x, const float* w, const float* y, int act, float* dy, float* dx,
                     int x_act, float* dx_colsum, float* dw, float* dbias, void* ws, size_t ws_bytes,
                     void* cuda_stream) {
    return fc_bwd_impl(N, C, K, x, w, y, act, dy, dx, x_act, dx_colsum, dw, dbias, ws, ws_bytes, cuda_stream);
}

int pcl_fc_bwd_fused_sgd(int N, int C, int K, const float* x, float* w, const float* y, int act, float* dy, float* dx,
                         int x_act, float* dx_colsum, float lr, float* dbias, void* ws, size_t ws_bytes,
                         void* cuda_stream) {
    if (!w) return PCL_ERR_BAD_ARG;
    return fc_bwd_impl(N, C, K, x, w, y, act, dy, dx, x_act, dx_colsum, nullptr, dbias, ws, ws_bytes, cuda_stream, w, lr);
}

size_t pcl_fc_bwd_fused_sgd_workspace_bytes(int N, int C, int K) {
    if (N <= 0 || C <= 0 || K <= 0) return 0;
    const pcl_conv_desc d{N, C, K, 1, 1, 1, 1, 1, 1, 0, 0};
    // (sized for either form of the weight-gradient part, like pcl_fc_workspace_bytes)
    const size_t wgrad_form = pcl_conv_bwd_weights_sgd_workspace_bytes(&d);
    const size_t fwd_form = fc_dzt_bytes(N, K) + plan_wgrad(d, 1, 1).colsum_bytes;
    return pcl_conv_bwd_data_colsum_workspace_bytes(&d) + align_up(wgrad_form > fwd_form ? wgrad_form : fwd_form, 256);
}

int pcl_plan_cache_stats(unsigned long long* hits, unsigned long long* misses) {
    plan_cache_stats(hits, misses);
    return PCL_OK;
}

int pcl_sgd_update(float* w, const float* dw, size_t n, float lr, void* cuda_stream) {
    if (!w || !dw) return n == 0 ? PCL_OK : PCL_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(dw)) & 3) return PCL_ERR_MISALIGNED;
    return launch_sgd(w, dw, n, lr, static_cast<cudaStream_t>(cuda_stream));
}

int pcl_maxpool2x2_fwd(int N, int H, int W, int C, const float* x, float* y, void* cuda_stream) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !x || !y) return PCL_ERR_BAD_ARG;
    if ((H | W) & 1) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return PCL_ERR_MISALIGNED;
    return launch_maxpool_fwd(N, H, W, C, x, y, static_cast<cudaStream_t>(cuda_stream));
}

int pcl_maxpool2x2_bwd(int N, int H, int W, int C, const float* x, const float* dy, const float* relu_mask_src,
                       float* dx, void* cuda_stream) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || !x || !dy || !dx) return PCL_ERR_BAD_ARG;
    if ((H | W) & 1) return PCL_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(relu_mask_src)) return PCL_ERR_MISALIGNED;
    return launch_maxpool_bwd(N, H, W, C, x, dy, relu_mask_src, dx, static_cast<cudaStream_t>(cuda_stream));
}

int pcl_softmax_xent(int N, int K, const float* logits, const int* labels, float* loss, float* dlogits,
                     void* cuda_stream) {
    if (N <= 0 || K <= 0 || !logits || !labels || !loss || !dlogits) return PCL_ERR_BAD_ARG;
    return launch_softmax_xent(N, K, logits, labels, loss, dlogits, static_cast<cudaStream_t>(cuda_stream));
}

static std::atomic<unsigned int> g_last_wait_code{0};

int pcl_last_device_status(void* cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return PCL_ERR_CUDA;
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)) != cudaSuccess) return PCL_ERR_CUDA;      // word [0]
    if (v != 0) {
        g_last_wait_code.store(v);
        const unsigned int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return PCL_ERR_CUDA;
        return v == kStatusBadLabel ? PCL_ERR_BAD_LABEL : PCL_ERR_DEVICE_TIMEOUT;
    }
    return PCL_OK;
}

unsigned int pcl_last_wait_code(void) { return g_last_wait_code.load(); }

unsigned long long pcl_launch_count(void) { return g_launches.load(); }

int pcl_profile_begin(void) {
    std::lock_guard<std::mutex> lock(g_prof_mu);
    g_prof_entries.clear();
    g_prof_pool_used = 0;
    g_prof_on = true;
    return PCL_OK;
}

int pcl_profile_end(pcl_kernel_stat* stats, int max_stats, int* n_stats) {
    if (!stats || !n_stats || max_stats < 0) return PCL_ERR_BAD_ARG;
    std::lock_guard<std::mutex> lock(g_prof_mu);
    g_prof_on = false;
    static pcl_kernel_stat agg[PROF_PASS_COUNT * KID_COUNT];
    memset(agg, 0, sizeof(agg));
    int rc = PCL_OK;
    for (const ProfEntry& e : g_prof_entries) {
        float ms = 0.f;
        if (cudaEventSynchronize(e.e1) != cudaSuccess || cudaEventElapsedTime(&ms, e.e0, e.e1) != cudaSuccess) {
            rc = PCL_ERR_CUDA;
            break;
        }
        pcl_kernel_stat& a = agg[e.pass * KID_COUNT + e.kid];
        a.launches += 1;
        a.total_ms += ms;
        a.work += e.work;
    }
    g_prof_entries.clear();
    g_prof_pool_used = 0;
    int n = 0;
    for (int k = 0; k < PROF_PASS_COUNT * KID_COUNT && n < max_stats; ++k) {
        if (agg[k].launches == 0) continue;
        snprintf(agg[k].name, sizeof(agg[k].name), "%s/%s", kPassNames[k / KID_COUNT], kKernelNames[k % KID_COUNT]);
        stats[n++] = agg[k];
    }
    *n_stats = n;
    return rc;
}

const char* pcl_status_string(int status) {
    switch (status) {
        case PCL_OK: return "ok";
        case PCL_ERR_BAD_ARG: return "bad argument";
        case PCL_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case PCL_ERR_MISALIGNED: return "misaligned pointer";
        case PCL_ERR_WORKSPACE: return "workspace too small";
        case PCL_ERR_CUDA: return "CUDA call failed";
        case PCL_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case PCL_ERR_SCRATCH_LIMIT: return "problem exceeds the capacity of the built-in scratch array";
        case PCL_ERR_BAD_LABEL: return "a class label lies outside [0, K)";
    }
    return "unknown status";
}

}  // extern "C"
