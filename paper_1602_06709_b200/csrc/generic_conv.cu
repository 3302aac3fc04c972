// Generic CUDA-core (fp32 FFMA) implicit-GEMM kernels for the three convolution
// passes.  They take any stride, padding and channel count, and serve the layers
// the tensor-core kernels do not cover (3-channel first layers, strided layers).
//
// One shared-memory tiled GEMM (64 x 64 x 16 tile, 256 threads, 4 x 4 outputs
// per thread); the three passes differ only in how a (row, reduction index) or
// (column, reduction index) pair maps to a tensor element:
//   forward       rows = output pixels (n,p,q), cols = k, reduction = (r,s,c)   Algorithm 1
//   backward-data rows = input pixels (n,h,w),  cols = c, reduction = (r,s,k)   gather form
//   weight-grad   rows = k, cols = (r,s,c), reduction = output pixels (n,p,q), split over CTAs
#include "pcl_internal.h"

namespace pcl {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

struct ConvGeom {
    int N, C, K, H, W, R, S, sh, sw, ph, pw, P, Q;
};

struct FwdProblem {
    ConvGeom g;
    const float *x, *w, *bias;
    float* y;
    int act;
    __device__ long rows() const { return long(g.N) * g.P * g.Q; }
    __device__ long cols() const { return g.K; }
    __device__ long depth() const { return long(g.R) * g.S * g.C; }
    __device__ float a(long m, long kk) const {
        const int q = int(m % g.Q); m /= g.Q;
        const int p = int(m % g.P); const long n = m / g.P;
        const int c = int(kk % g.C); const int tap = int(kk / g.C);
        const int s = tap % g.S, r = tap / g.S;
        const int h = p * g.sh + r - g.ph, ww = q * g.sw + s - g.pw;
        if (h < 0 || h >= g.H || ww < 0 || ww >= g.W) return 0.f;
        return __ldg(x + ((n * g.H + h) * g.W + ww) * g.C + c);
    }
    __device__ float b(long col, long kk) const { return __ldg(w + col * depth() + kk); }
    __device__ void store(long m, long col, float v, int) const {
        if (bias) v += __ldg(bias + col);
        if (act == PCL_ACT_RELU) v = fmaxf(v, 0.f);
        else if (act == PCL_ACT_SIGMOID) v = sigmoid_fast(v);
        y[m * g.K + col] = v;
    }
};

struct DgradProblem {
    ConvGeom g;
    const float *dy, *w, *mask;
    float* dx;
    __device__ long rows() const { return long(g.N) * g.H * g.W; }
    __device__ long cols() const { return g.C; }
    __device__ long depth() const { return long(g.R) * g.S * g.K; }
    __device__ float a(long m, long kk) const {
        const int ww = int(m % g.W); m /= g.W;
        const int h = int(m % g.H); const long n = m / g.H;
        const int k = int(kk % g.K); const int tap = int(kk / g.K);
        const int s = tap % g.S, r = tap / g.S;
        const int hp = h + g.ph - r, wq = ww + g.pw - s;
        if (hp < 0 || wq < 0 || hp % g.sh != 0 || wq % g.sw != 0) return 0.f;
        const int p = hp / g.sh, q = wq / g.sw;
        if (p >= g.P || q >= g.Q) return 0.f;
        return __ldg(dy + ((n * g.P + p) * g.Q + q) * g.K + k);
    }
    __device__ float b(long col, long kk) const {
        const int k = int(kk % g.K); const int tap = int(kk / g.K);
        return __ldg(w + (long(k) * g.R * g.S + tap) * g.C + col);
    }
    __device__ void store(long m, long col, float v, int) const {
        const long i = m * g.C + col;
        if (mask && !(__ldg(mask + i) > 0.f)) v = 0.f;
        dx[i] = v;
    }
};

struct WgradProblem {
    ConvGeom g;
    const float *x, *dy;
    float* out;            // dw or partial workspace
    size_t split_stride;
    __device__ long rows() const { return g.K; }
    __device__ long cols() const { return long(g.R) * g.S * g.C; }
    __device__ long depth() const { return long(g.N) * g.P * g.Q; }
    __device__ float a(long k, long kk) const { return __ldg(dy + kk * g.K + k); }
    __device__ float b(long col, long kk) const {
        const int c = int(col % g.C); const int tap = int(col / g.C);
        const int s = tap % g.S, r = tap / g.S;
        const int q = int(kk % g.Q); kk /= g.Q;
        const int p = int(kk % g.P); const long n = kk / g.P;
        const int h = p * g.sh + r - g.ph, ww = q * g.sw + s - g.pw;
        if (h < 0 || h >= g.H || ww < 0 || ww >= g.W) return 0.f;
        return __ldg(x + ((n * g.H + h) * g.W + ww) * g.C + c);
    }
    __device__ void store(long k, long col, float v, int split) const {
        out[size_t(split) * split_stride + k * cols() + col] = v;
    }
};

template <class Problem>
__global__ void __launch_bounds__(256) generic_gemm_kernel(Problem pr, long depth_per_split) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const long row0 = long(blockIdx.x) * BM, col0 = long(blockIdx.y) * BN;
    const int split = blockIdx.z;
    const long d_begin = split * depth_per_split;
    long d_end = d_begin + depth_per_split;
    if (d_end > pr.depth()) d_end = pr.depth();
    const long M = pr.rows(), Nc = pr.cols();

    const int lrow = tid >> 2, lk = (tid & 3) * 4;     // loader: one row, 4 consecutive reduction indices
    const int ty = tid >> 4, tx = tid & 15;            // compute: 4 x 4 outputs at (ty*4, tx*4)
    float acc[4][4] = {};

    for (long d0 = d_begin; d0 < d_end; d0 += BK) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long kk = d0 + lk + j;
            const long ra = row0 + lrow, cb = col0 + lrow;
            As[lk + j][lrow] = (kk < d_end && ra < M) ? pr.a(ra, kk) : 0.f;
            Bs[lk + j][lrow] = (kk < d_end && cb < Nc) ? pr.b(cb, kk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a4[4] = {av.x, av.y, av.z, av.w};
            const float b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a4[i], b4[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long r = row0 + ty * 4 + i, c = col0 + tx * 4 + j;
            if (r < M && c < Nc) pr.store(r, c, acc[i][j], split);
        }
}

ConvGeom geom(const pcl_conv_desc& d, int P, int Q) {
    return ConvGeom{d.N, d.C, d.K, d.H, d.W, d.R, d.S, d.stride_h, d.stride_w, d.pad_h, d.pad_w, P, Q};
}

template <class Problem>
int launch(const Problem& pr, int kid, long rows, long cols, long depth, int splits, cudaStream_t st) {
    const long gx = (rows + BM - 1) / BM, gy = (cols + BN - 1) / BN;
    if (gx > 0x7fffffffL || gy > 65535 || splits > 65535) return PCL_ERR_UNSUPPORTED_SHAPE;
    long per = (depth + splits - 1) / splits;
    per = (per + BK - 1) / BK * BK;
    {
        LaunchScope scope(kid, 2.0 * double(rows) * double(cols) * double(depth), st);
        generic_gemm_kernel<Problem><<<dim3(unsigned(gx), unsigned(gy), unsigned(splits)), 256, 0, st>>>(pr, per);
    }
    return cudaGetLastError() == cudaSuccess ? PCL_OK : PCL_ERR_CUDA;
}

}  // namespace

int launch_generic_fwd(const pcl_conv_desc& d, int P, int Q, const float* x, const float* w, const float* bias,
                       float* y, int act, cudaStream_t st) {
    FwdProblem pr{geom(d, P, Q), x, w, bias, y, act};
    return launch(pr, KID_GENERIC_FWD, long(d.N) * P * Q, d.K, long(d.R) * d.S * d.C, 1, st);
}

int launch_generic_bwd_data(const pcl_conv_desc& d, int P, int Q, const float* dy, const float* w,
                            const float* mask_src, float* dx, cudaStream_t st) {
    DgradProblem pr{geom(d, P, Q), dy, w, mask_src, dx};
    return launch(pr, KID_GENERIC_DGRAD, long(d.N) * d.H * d.W, d.C, long(d.R) * d.S * d.K, 1, st);
}

int generic_wgrad_splits(const pcl_conv_desc& d, int P, int Q) {
    const long tiles = long((d.K + BM - 1) / BM) * ((long(d.R) * d.S * d.C + BN - 1) / BN);
    const long depth = long(d.N) * P * Q;
    long splits = (4 * device_sm_count() + tiles - 1) / tiles;
    const long max_by_depth = (depth + 255) / 256;
    if (splits > max_by_depth) splits = max_by_depth;
    if (splits > 256) splits = 256;
    if (splits < 1) splits = 1;
    long per = (depth + splits - 1) / splits;
    per = (per + BK - 1) / BK * BK;
    splits = (depth + per - 1) / per;
    return int(splits);
}

int launch_generic_bwd_weights(const pcl_conv_desc& d, int P, int Q, const float* x, const float* dy, float* dw,
                               float* partial, int splits, cudaStream_t st) {
    const size_t dw_elems = size_t(d.K) * d.R * d.S * d.C;
    if (splits > 1 && !partial) return PCL_ERR_WORKSPACE;
    WgradProblem pr{geom(d, P, Q), x, dy, splits > 1 ? partial : dw, splits > 1 ? dw_elems : 0};
    int rc = launch(pr, KID_GENERIC_WGRAD, d.K, long(d.R) * d.S * d.C, long(d.N) * P * Q, splits, st);
    if (rc != PCL_OK) return rc;
    if (splits > 1) return launch_reduce_splits(partial, dw, dw_elems, splits, st);
    return PCL_OK;
}

}  // namespace pcl
