// HBM-bound kernels: SGD update, split reduction, weight transpose, activation
// gradient, column sums, 2x2 max-pool, softmax cross-entropy.  All are plain
// coalesced, vectorised (float4 where alignment allows) grid-stride kernels;
// their roofline is memory bandwidth.
#include <math.h>

#include "pcl_internal.h"

namespace pcl {

namespace {

int grid_for(size_t work_items, int block, int per_sm = 8) {
    size_t blocks = (work_items + block - 1) / block;
    const size_t cap = size_t(device_sm_count()) * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return int(blocks);
}

// w <- w - lr * dw.  12 bytes of traffic per parameter.
__global__ void __launch_bounds__(256) sgd_kernel(float* __restrict__ w, const float* __restrict__ dw, size_t n,
                                                  float lr, int vec) {
    const size_t tid = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    if (vec) {
        const size_t n4 = n >> 2;
        float4* w4 = reinterpret_cast<float4*>(w);
        const float4* d4 = reinterpret_cast<const float4*>(dw);
        for (size_t i = tid; i < n4; i += stride) {
            float4 a = w4[i];
            const float4 g = __ldcs(d4 + i);
            a.x = fmaf(-lr, g.x, a.x); a.y = fmaf(-lr, g.y, a.y);
            a.z = fmaf(-lr, g.z, a.z); a.w = fmaf(-lr, g.w, a.w);
            w4[i] = a;
        }
        for (size_t i = (n4 << 2) + tid; i < n; i += stride) w[i] = fmaf(-lr, dw[i], w[i]);
    } else {
        for (size_t i = tid; i < n; i += stride) w[i] = fmaf(-lr, dw[i], w[i]);
    }
}

__global__ void __launch_bounds__(256) zero_kernel(float* __restrict__ p, size_t n) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) p[i] = 0.f;
}

// out[i] = partial[0][i] + partial[1][i] + ... in that order (fixed => reproducible)
__global__ void __launch_bounds__(256) reduce_splits_kernel(const float* __restrict__ partial, float* __restrict__ out,
                                                            size_t n, int splits) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        float acc = partial[i];
        for (int s = 1; s < splits; ++s) acc += partial[size_t(s) * n + i];
        out[i] = acc;
    }
}

// w[i] <- w[i] - lr * (partial[0][i] + partial[1][i] + ...): the weight gradient's second pass applying the update itself
// (Sec. 3.1: a layer's new weights are not needed before its next forward pass).  The sum is formed exactly as
// reduce_splits_kernel forms it and applied exactly as sgd_kernel applies it, so the result equals the two-kernel form bit
// for bit; dw itself is never written.
__global__ void __launch_bounds__(256) reduce_splits_sgd_kernel(const float* __restrict__ partial, float* __restrict__ w,
                                                                size_t n, int splits, float lr) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        float acc = partial[i];
        for (int s = 1; s < splits; ++s) acc += partial[size_t(s) * n + i];
        w[i] = fmaf(-lr, acc, w[i]);
    }
}

// wt_t[c][R-1-r][S-1-s][k] = w[k][r][s][c]: the "transpose-weights" copy the
// backward-data pass contracts against (Sec. 2.3 keeps such a copy too).
__global__ void __launch_bounds__(256) transpose_flip_kernel(const float* __restrict__ w, float* __restrict__ out,
                                                             int K, int RS, int C) {
    __shared__ float tile[32][33];
    const int tap = blockIdx.z;
    const int k0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
    for (int j = ty; j < 32; j += 8) {
        const int k = k0 + j, c = c0 + tx;
        tile[j][tx] = (k < K && c < C) ? w[(size_t(k) * RS + tap) * C + c] : 0.f;
    }
    __syncthreads();
    const int tap_f = RS - 1 - tap;   // flipping r and s together reverses the flat tap index
    for (int j = ty; j < 32; j += 8) {
        const int c = c0 + j, k = k0 + tx;
        if (k < K && c < C) out[(size_t(c) * RS + tap_f) * K + k] = tile[tx][j];
    }
}

__global__ void __launch_bounds__(256) act_grad_kernel(float* __restrict__ dy, const float* __restrict__ y, size_t n,
                                                       int act) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float yv = y[i];
        const float g = dy[i];
        dy[i] = act == PCL_ACT_RELU ? (yv > 0.f ? g : 0.f) : g * yv * (1.f - yv);
    }
}

// partial[split][k] = sum over the split's rows of m[row][k].
// A block covers a strip of up to 1024 columns (256 threads x float4 when K is a
// multiple of 4) so that consecutive rows are read as whole contiguous runs; the
// threads that share a column group are summed through shared memory in a fixed order.
constexpr int kColsumMinRows = 64;     // rows per split, at least; grown so that there are at most ~1200 splits
template <int VEC>
__global__ void __launch_bounds__(256) colsum_kernel(const float* __restrict__ m, size_t rows, int K,
                                                     float* __restrict__ partial, size_t rows_per_split, int strip) {
    const int kv = K / VEC;                                  // column groups per row
    // strip: column groups this block covers per row (see colsum_strip())
    const int lanes = 256 / strip;                           // rows handled concurrently
    const int cg = blockIdx.x * strip + threadIdx.x % strip; // this thread's column group
    const int rl = threadIdx.x / strip;
    const size_t r0 = size_t(blockIdx.y) * rows_per_split;
    size_t r1 = r0 + rows_per_split;
    if (r1 > rows) r1 = rows;
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    if (cg < kv && rl < lanes) {
        size_t r = r0 + rl;
        for (; r + 3 * size_t(lanes) < r1; r += 4 * size_t(lanes)) {      // 4 independent loads in flight
            float t[4][VEC];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float* src = m + (r + u * size_t(lanes)) * K + size_t(cg) * VEC;
                if (VEC == 4) {
                    const float4 q = __ldcs(reinterpret_cast<const float4*>(src));
                    t[u][0] = q.x; t[u][1 % VEC] = q.y; t[u][2 % VEC] = q.z; t[u][3 % VEC] = q.w;
                } else {
                    t[u][0] = __ldcs(src);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[v] += t[u][v];
        }
        for (; r < r1; r += lanes) {
            const float* src = m + r * K + size_t(cg) * VEC;
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] += src[v];
        }
    }
    __shared__ float red[256][VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) red[threadIdx.x][v] = acc[v];
    __syncthreads();
    if (rl == 0 && cg < kv) {
        for (int l = 1; l < lanes; ++l)
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] += red[threadIdx.x + l * strip][v];
#pragma unroll
        for (int v = 0; v < VEC; ++v) partial[size_t(blockIdx.y) * K + size_t(cg) * VEC + v] = acc[v];
    }
}

// Position code of a 2x2 window (a b / c d): bits 0-1 = position of the first maximum in row-major order, bit 2 set
// where that maximum is <= 0 (what a ReLU mask on the pooled layer would zero).
__device__ __forceinline__ unsigned int pool_code1(float a, float b, float c, float d) {
    unsigned int arg = 0; float best = a;
    if (b > best) { best = b; arg = 1; }
    if (c > best) { best = c; arg = 2; }
    if (d > best) { best = d; arg = 3; }
    return arg | (best > 0.f ? 0u : 4u);
}

// 2x2 / stride-2 max pooling, NHWC, one thread per (output pixel, 4 channels)
template <int VEC>
__global__ void __launch_bounds__(256) maxpool_fwd_kernel(const float* __restrict__ x, float* __restrict__ y, int N,
                                                          int H, int W, int C, unsigned char* __restrict__ idx = nullptr) {
    const int Po = H / 2, Qo = W / 2, Cv = C / VEC;
    const size_t total = size_t(N) * Po * Qo * Cv;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int cv = int(i % Cv); size_t t = i / Cv;
        const int q = int(t % Qo); t /= Qo;
        const int p = int(t % Po); const size_t n = t / Po;
        const float* src = x + ((n * H + 2 * p) * W + 2 * q) * C + cv * VEC;
        float* dst = y + ((n * Po + p) * Qo + q) * C + cv * VEC;
        if (VEC == 4) {
            const float4 a = *reinterpret_cast<const float4*>(src);
            const float4 b = *reinterpret_cast<const float4*>(src + C);
            const float4 c = *reinterpret_cast<const float4*>(src + size_t(W) * C);
            const float4 d = *reinterpret_cast<const float4*>(src + size_t(W) * C + C);
            float4 o;
            o.x = fmaxf(fmaxf(a.x, b.x), fmaxf(c.x, d.x)); o.y = fmaxf(fmaxf(a.y, b.y), fmaxf(c.y, d.y));
            o.z = fmaxf(fmaxf(a.z, b.z), fmaxf(c.z, d.z)); o.w = fmaxf(fmaxf(a.w, b.w), fmaxf(c.w, d.w));
            *reinterpret_cast<float4*>(dst) = o;
            if (idx) {
                unsigned int code = pool_code1(a.x, b.x, c.x, d.x) | (pool_code1(a.y, b.y, c.y, d.y) << 8) |
                                    (pool_code1(a.z, b.z, c.z, d.z) << 16) | (pool_code1(a.w, b.w, c.w, d.w) << 24);
                *reinterpret_cast<unsigned int*>(idx + (dst - y)) = code;
            }
        } else {
            dst[0] = fmaxf(fmaxf(src[0], src[C]), fmaxf(src[size_t(W) * C], src[size_t(W) * C + C]));
            if (idx) idx[dst - y] = static_cast<unsigned char>(pool_code1(src[0], src[C], src[size_t(W) * C], src[size_t(W) * C + C]));
        }
    }
}

__device__ __forceinline__ void pool_route(float a, float b, float c, float d, float g, float& oa, float& ob,
                                           float& oc, float& od) {
    // first maximum in row-major window order
    int arg = 0; float best = a;
    if (b > best) { best = b; arg = 1; }
    if (c > best) { best = c; arg = 2; }
    if (d > best) { best = d; arg = 3; }
    oa = arg == 0 ? g : 0.f; ob = arg == 1 ? g : 0.f; oc = arg == 2 ? g : 0.f; od = arg == 3 ? g : 0.f;
}

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 mask4(float4 v, float4 m) {
    return make_float4(m.x > 0.f ? v.x : 0.f, m.y > 0.f ? v.y : 0.f, m.z > 0.f ? v.z : 0.f, m.w > 0.f ? v.w : 0.f);
}

// One thread per (pooled pixel, VEC channels): reads the 2x2 window of x and one dy, writes the 2x2 window of
// dx.  When the ReLU mask source is x itself (the usual case: x is a ReLU output) it is not read again.
// colsum_rows (VEC == 4 only, C/4 must divide 256): row blockIdx.x receives the per-channel sums of everything this
// block wrote to dx.  Every thread keeps the same 4 channels for the whole grid-stride loop, so it sums privately;
// the threads of a block that share channels are then added in a fixed order.
template <int VEC>
__global__ void __launch_bounds__(256) maxpool_bwd_kernel(const float* __restrict__ x, const float* __restrict__ dy,
                                                          const float* __restrict__ mask, float* __restrict__ dx,
                                                          int N, int H, int W, int C,
                                                          float* __restrict__ colsum_rows = nullptr) {
    const int Po = H / 2, Qo = W / 2, Cv = C / VEC;
    const size_t total = size_t(N) * Po * Qo * Cv;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t rowp = size_t(W) * C;
    const bool mask_is_x = (mask == x);
    float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int cv = int(i % Cv); size_t t = i / Cv;
        const int q = int(t % Qo); t /= Qo;
        const int p = int(t % Po); const size_t n = t / Po;
        const size_t off = ((n * H + 2 * p) * W + 2 * q) * C + cv * VEC;
        const float* g = dy + ((n * Po + p) * Qo + q) * C + cv * VEC;
        if (VEC == 4) {
            const float4 a = ld4(x + off), b = ld4(x + off + C), c = ld4(x + off + rowp), d = ld4(x + off + rowp + C);
            const float4 gv = __ldcs(reinterpret_cast<const float4*>(g));
            float4 oa, ob, oc, od;
            pool_route(a.x, b.x, c.x, d.x, gv.x, oa.x, ob.x, oc.x, od.x);
            pool_route(a.y, b.y, c.y, d.y, gv.y, oa.y, ob.y, oc.y, od.y);
            pool_route(a.z, b.z, c.z, d.z, gv.z, oa.z, ob.z, oc.z, od.z);
            pool_route(a.w, b.w, c.w, d.w, gv.w, oa.w, ob.w, oc.w, od.w);
            if (mask) {
                if (mask_is_x) {
                    oa = mask4(oa, a); ob = mask4(ob, b); oc = mask4(oc, c); od = mask4(od, d);
                } else {
                    oa = mask4(oa, ld4(mask + off)); ob = mask4(ob, ld4(mask + off + C));
                    oc = mask4(oc, ld4(mask + off + rowp)); od = mask4(od, ld4(mask + off + rowp + C));
                }
            }
            __stcs(reinterpret_cast<float4*>(dx + off), oa);
            __stcs(reinterpret_cast<float4*>(dx + off + C), ob);
            __stcs(reinterpret_cast<float4*>(dx + off + rowp), oc);
            __stcs(reinterpret_cast<float4*>(dx + off + rowp + C), od);
            csum.x += (oa.x + ob.x) + (oc.x + od.x); csum.y += (oa.y + ob.y) + (oc.y + od.y);
            csum.z += (oa.z + ob.z) + (oc.z + od.z); csum.w += (oa.w + ob.w) + (oc.w + od.w);
        } else {
            const float a = x[off], b = x[off + C], c = x[off + rowp], d = x[off + rowp + C];
            float oa, ob, oc, od;
            pool_route(a, b, c, d, g[0], oa, ob, oc, od);
            if (mask) {
                if (!(mask[off] > 0.f)) oa = 0.f;
                if (!(mask[off + C] > 0.f)) ob = 0.f;
                if (!(mask[off + rowp] > 0.f)) oc = 0.f;
                if (!(mask[off + rowp + C] > 0.f)) od = 0.f;
            }
            dx[off] = oa; dx[off + C] = ob; dx[off + rowp] = oc; dx[off + rowp + C] = od;
        }
    }
    if (VEC == 4 && colsum_rows) {
        __shared__ float4 red[256];
        red[threadIdx.x] = csum;
        __syncthreads();
        const int Cv4 = C / 4;
        if (threadIdx.x < Cv4) {
            float4 a = red[threadIdx.x];
            for (int t = threadIdx.x + Cv4; t < 256; t += Cv4) {
                a.x += red[t].x; a.y += red[t].y; a.z += red[t].z; a.w += red[t].w;
            }
            *reinterpret_cast<float4*>(colsum_rows + size_t(blockIdx.x) * C + threadIdx.x * 4) = a;
        }
    }
}

// Pooling backward from the position codes the forward pass recorded (no pass over the pooled layer's input):
// dx gets dy at the coded position of each window and 0 elsewhere; with `relu`, windows whose code has bit 2 set
// (maximum <= 0) get 0 everywhere.  Column sums as in maxpool_bwd_kernel.
template <int VEC>
__global__ void __launch_bounds__(256) maxpool_bwd_idx_kernel(const unsigned char* __restrict__ idx,
                                                              const float* __restrict__ dy, int relu,
                                                              float* __restrict__ dx, int N, int H, int W, int C,
                                                              float* __restrict__ colsum_rows = nullptr) {
    const int Po = H / 2, Qo = W / 2, Cv = C / VEC;
    const size_t total = size_t(N) * Po * Qo * Cv;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    const size_t rowp = size_t(W) * C;
    const unsigned int kill = relu ? 4u : 0u;
    float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int cv = int(i % Cv); size_t t = i / Cv;
        const int q = int(t % Qo); t /= Qo;
        const int p = int(t % Po); const size_t n = t / Po;
        const size_t off = ((n * H + 2 * p) * W + 2 * q) * C + cv * VEC;
        const size_t po = ((n * Po + p) * Qo + q) * C + cv * VEC;
        if (VEC == 4) {
            const float4 gv = __ldcs(reinterpret_cast<const float4*>(dy + po));
            const unsigned int code = __ldcs(reinterpret_cast<const unsigned int*>(idx + po));
            const float g[4] = {gv.x, gv.y, gv.z, gv.w};
            float o[4][4];      // [position][channel]
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const unsigned int cc = (code >> (8 * c)) & 0xffu;
                const float gg = (cc & kill) ? 0.f : g[c];
#pragma unroll
                for (int e = 0; e < 4; ++e) o[e][c] = (cc & 3u) == unsigned(e) ? gg : 0.f;
                (&csum.x)[c] += gg;
            }
            __stcs(reinterpret_cast<float4*>(dx + off), make_float4(o[0][0], o[0][1], o[0][2], o[0][3]));
            __stcs(reinterpret_cast<float4*>(dx + off + C), make_float4(o[1][0], o[1][1], o[1][2], o[1][3]));
            __stcs(reinterpret_cast<float4*>(dx + off + rowp), make_float4(o[2][0], o[2][1], o[2][2], o[2][3]));
            __stcs(reinterpret_cast<float4*>(dx + off + rowp + C), make_float4(o[3][0], o[3][1], o[3][2], o[3][3]));
        } else {
            const unsigned int cc = idx[po];
            const float gg = (cc & kill) ? 0.f : dy[po];
            dx[off] = (cc & 3u) == 0u ? gg : 0.f;
            dx[off + C] = (cc & 3u) == 1u ? gg : 0.f;
            dx[off + rowp] = (cc & 3u) == 2u ? gg : 0.f;
            dx[off + rowp + C] = (cc & 3u) == 3u ? gg : 0.f;
        }
    }
    if (VEC == 4 && colsum_rows) {
        __shared__ float4 red[256];
        red[threadIdx.x] = csum;
        __syncthreads();
        const int Cv4 = C / 4;
        if (threadIdx.x < Cv4) {
            float4 a = red[threadIdx.x];
            for (int t = threadIdx.x + Cv4; t < 256; t += Cv4) {
                a.x += red[t].x; a.y += red[t].y; a.z += red[t].z; a.w += red[t].w;
            }
            *reinterpret_cast<float4*>(colsum_rows + size_t(blockIdx.x) * C + threadIdx.x * 4) = a;
        }
    }
}

// One CTA per row: max, sum of exponentials, loss term, gradient.
__global__ void __launch_bounds__(256) softmax_xent_kernel(const float* __restrict__ logits,
                                                           const int* __restrict__ labels, float* __restrict__ loss,
                                                           float* __restrict__ dlogits, int N, int K,
                                                           unsigned int* __restrict__ status) {
    __shared__ float red[32];
    __shared__ float bcast;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        const float* z = logits + size_t(n) * K;
        float mx = -INFINITY;
        for (int k = threadIdx.x; k < K; k += blockDim.x) mx = fmaxf(mx, z[k]);
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) red[warp] = mx;
        __syncthreads();
        if (warp == 0) {
            float v = lane < (blockDim.x >> 5) ? red[lane] : -INFINITY;
            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (lane == 0) bcast = v;
        }
        __syncthreads();
        mx = bcast;
        float sum = 0.f;
        for (int k = threadIdx.x; k < K; k += blockDim.x) sum += expf(z[k] - mx);
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        __syncthreads();
        if (lane == 0) red[warp] = sum;
        __syncthreads();
        if (warp == 0) {
            float v = lane < (blockDim.x >> 5) ? red[lane] : 0.f;
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) bcast = v;
        }
        __syncthreads();
        sum = bcast;
        // a label outside [0, K) names no class: the row gets no target and no loss term (nothing is read through
        // it), and the device status word records it
        int lab = labels[n];
        if (lab < 0 || lab >= K) {
            if (threadIdx.x == 0) atomicCAS(status, 0u, static_cast<unsigned int>(kStatusBadLabel));
            lab = -1;
        }
        const float inv_n = 1.f / float(N);
        const float inv_sum = 1.f / sum;
        for (int k = threadIdx.x; k < K; k += blockDim.x) {
            const float pk = expf(z[k] - mx) * inv_sum;
            dlogits[size_t(n) * K + k] = (pk - (k == lab ? 1.f : 0.f)) * inv_n;
        }
        if (threadIdx.x == 0 && lab >= 0) atomicAdd(loss, -(z[lab] - mx - logf(sum)) * inv_n);
        __syncthreads();
    }
}

// The same for rows of at most 256 * kPer values: the row is read once and kept in registers (the three passes of the
// kernel above re-read it from L1/L2), thread t holding elements t, t + 256, ...
// kVec = 4 (K % 4 == 0, 16-byte aligned rows): thread t holds elements 4 * (256 * j + t) .. + 3, read and written as
// float4; kVec = 1: elements 256 * i + t.  The exponentials are ex2.approx of the scaled argument (arguments in
// [-|row range|, 0]: relative error ~1e-6, well inside the 1e-4 the gradients are held to).
template <int kPer, int kVec>
__global__ void __launch_bounds__(256) softmax_xent_regs_kernel(const float* __restrict__ logits,
                                                                const int* __restrict__ labels, float* __restrict__ loss,
                                                                float* __restrict__ dlogits, int N, int K,
                                                                unsigned int* __restrict__ status) {
    __shared__ float red[8];
    __shared__ float bcast;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // index of this thread's i-th element in the row
    auto elem = [](int i) { return kVec == 4 ? 4 * (256 * (i >> 2) + int(threadIdx.x)) + (i & 3) : i * 256 + int(threadIdx.x); };
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        const float* z = logits + size_t(n) * K;
        float v[kPer];
        float mx = -INFINITY;
        if (kVec == 4) {
#pragma unroll
            for (int j = 0; j < kPer / 4; ++j) {
                const int k = elem(4 * j);
                float4 q = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                if (k < K) q = __ldg(reinterpret_cast<const float4*>(z + k));
                v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
                mx = fmaxf(fmaxf(mx, fmaxf(q.x, q.y)), fmaxf(q.z, q.w));
            }
        } else {
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const int k = elem(i);
                v[i] = k < K ? __ldg(z + k) : -INFINITY;
                mx = fmaxf(mx, v[i]);
            }
        }
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) red[warp] = mx;
        __syncthreads();
        if (warp == 0) {
            float t = lane < 8 ? red[lane] : -INFINITY;
            for (int o = 4; o > 0; o >>= 1) t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, o));
            if (lane == 0) bcast = t;
        }
        __syncthreads();
        mx = bcast;
        int lab = labels[n];
        if (lab < 0 || lab >= K) {
            if (threadIdx.x == 0) atomicCAS(status, 0u, static_cast<unsigned int>(kStatusBadLabel));
            lab = -1;
        }
        float sum = 0.f, zlab = 0.f;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int k = elem(i);
            if (k == lab) zlab = v[i];
            v[i] = k < K ? __expf(v[i] - mx) : 0.f;
            sum += v[i];
        }
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        __syncthreads();
        if (lane == 0) red[warp] = sum;
        __syncthreads();
        if (warp == 0) {
            float t = lane < 8 ? red[lane] : 0.f;
            for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) bcast = t;
        }
        __syncthreads();
        sum = bcast;
        const float inv_n = 1.f / float(N), inv_sum = 1.f / sum;
        float* out = dlogits + size_t(n) * K;
        if (kVec == 4) {
#pragma unroll
            for (int j = 0; j < kPer / 4; ++j) {
                const int k = elem(4 * j);
                if (k < K)
                    *reinterpret_cast<float4*>(out + k) = make_float4((v[4 * j] * inv_sum - (k == lab ? 1.f : 0.f)) * inv_n,
                                                                      (v[4 * j + 1] * inv_sum - (k + 1 == lab ? 1.f : 0.f)) * inv_n,
                                                                      (v[4 * j + 2] * inv_sum - (k + 2 == lab ? 1.f : 0.f)) * inv_n,
                                                                      (v[4 * j + 3] * inv_sum - (k + 3 == lab ? 1.f : 0.f)) * inv_n);
            }
        } else {
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const int k = elem(i);
                if (k < K) out[k] = (v[i] * inv_sum - (k == lab ? 1.f : 0.f)) * inv_n;
            }
        }
        // (the thread that holds the labelled element adds the row's loss term)
        const int owner = kVec == 4 ? (lab >> 2) & 255 : lab & 255;
        if (lab >= 0 && owner == int(threadIdx.x)) atomicAdd(loss, -(zlab - mx - logf(sum)) * inv_n);
        __syncthreads();
    }
}

// xs[n][hh][ww][0..3]: channel-padded, TF32-rounded copy of x with a zero halo of (pad_h, pad_w).  One block per padded image row
// (no per-pixel index divisions: the kernel is otherwise bound by them, not by memory); the block after the last
// row writes the trailing zero pixels (windows are read 32 floats wide, so the last ones reach past the last row).
__global__ void __launch_bounds__(256) stage_pad_c4_kernel(const float* __restrict__ x, float4* __restrict__ xs, int N,
                                                           int H, int W, int C, int pad_h, int pad_w, int slack) {
    const int Hp = H + 2 * pad_h, Wp = W + 2 * pad_w;
    const size_t row = blockIdx.x;                       // n * Hp + hh + pad_h
    if (row == size_t(N) * Hp) {
        if (int(threadIdx.x) < slack) xs[row * Wp + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const size_t n = row / Hp;
    const int hh = int(row - n * Hp) - pad_h;
    float4* dst = xs + row * Wp;
    if (hh < 0 || hh >= H) {
        for (int i = threadIdx.x; i < Wp; i += blockDim.x) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const float* src = x + (n * H + hh) * size_t(W) * C;
    for (int i = threadIdx.x; i < Wp; i += blockDim.x) {
        const int ww = i - pad_w;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (ww >= 0 && ww < W)
            for (int c = 0; c < C; ++c) {
                // rounded to TF32 (nearest even) here, once: what a TMA load through a TFLOAT32 tensor map would do to
                // every element it fetches; the tensor-core kernels may then also copy the staged data with plain loads
                uint32_t r;
                asm("cvt.rn.tf32.f32 %0, %1;" : "=r"(r) : "f"(__ldg(src + size_t(ww) * C + c)));
                v[c] = __uint_as_float(r);
            }
        dst[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// w32[k*R + r][s*4 + c] = w[k][r][s][c] for c < C, s < S; every other element of the row_floats-long row is zero
__global__ void __launch_bounds__(256) stage_w4_kernel(const float* __restrict__ w, float* __restrict__ w32,
                                                       size_t rows, int S, int C, int row_floats) {
    const size_t total = rows * row_floats;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const size_t row = i / row_floats; const int j = int(i - row * row_floats);
        const int s = j >> 2, c = j & 3;
        w32[i] = (s < S && c < C) ? w[(row * S + s) * C + c] : 0.f;
    }
}

// dw[row][s][c] = sum over splits of dw4[split][row][s*4 + c], c < C, s < S  (fixed order)
__global__ void __launch_bounds__(256) unpad_reduce_kernel(const float* __restrict__ dw4, float* __restrict__ dw,
                                                           size_t rows, int S, int C, int row_floats, int splits,
                                                           size_t split_stride) {
    const size_t total = rows * S * C;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const size_t tap = i / C; const int c = int(i % C);
        const size_t row = tap / S; const int s = int(tap - row * S);
        float acc = 0.f;
        for (int sp = 0; sp < splits; ++sp) acc += dw4[size_t(sp) * split_stride + row * row_floats + s * 4 + c];
        dw[i] = acc;
    }
}

// One phase of a strided backward-data pass: out[c][Ra-1-i][Sb-1-j][k] = w[k][a + i*sh][b + j*sw][c].
__global__ void __launch_bounds__(256) phase_weights_kernel(const float* __restrict__ w, float* __restrict__ out, int K,
                                                            int R, int S, int C, int a, int b, int sh, int sw, int Ra,
                                                            int Sb) {
    const size_t total = size_t(C) * Ra * Sb * K;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t o = size_t(blockIdx.x) * blockDim.x + threadIdx.x; o < total; o += stride) {
        const int k = int(o % K); size_t t = o / K;
        const int jj = int(t % Sb); t /= Sb;
        const int ii = int(t % Ra); const int c = int(t / Ra);
        const int r = a + (Ra - 1 - ii) * sh, s = b + (Sb - 1 - jj) * sw;
        out[o] = w[((size_t(k) * R + r) * S + s) * C + c];
    }
}

#define PCL_CHECK_LAUNCH() (cudaGetLastError() == cudaSuccess ? PCL_OK : PCL_ERR_CUDA)

}  // namespace

int launch_sgd(float* w, const float* dw, size_t n, float lr, cudaStream_t st) {
    if (n == 0) return PCL_OK;
    const int vec = ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(dw)) & 15) == 0;
    {
        LaunchScope scope(KID_SGD, 12.0 * double(n), st);
        sgd_kernel<<<grid_for(vec ? (n + 3) / 4 : n, 256), 256, 0, st>>>(w, dw, n, lr, vec);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_zero(float* p, size_t n, cudaStream_t st) {
    if (n == 0) return PCL_OK;
    {
        LaunchScope scope(KID_ZERO, 4.0 * double(n), st);
        zero_kernel<<<grid_for(n, 256), 256, 0, st>>>(p, n);
    }
    return PCL_CHECK_LAUNCH();
}

// out[r][k] = act(bias[k] + sum_s partial[s][r][k]): second pass of a split-reduction forward-type launch
__global__ void __launch_bounds__(256) reduce_splits_bias_act_kernel(const float4* __restrict__ partial, float4* __restrict__ out,
                                                                      const float* __restrict__ bias, int act, size_t n4,
                                                                      int K4, int splits) {
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 acc = partial[i];
        for (int s = 1; s < splits; ++s) {
            const float4 v = partial[size_t(s) * n4 + i];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (bias) {
            const float4 b = __ldg(reinterpret_cast<const float4*>(bias) + (i % K4));
            acc.x += b.x; acc.y += b.y; acc.z += b.z; acc.w += b.w;
        }
        if (act == PCL_ACT_RELU) {
            acc.x = fmaxf(acc.x, 0.f); acc.y = fmaxf(acc.y, 0.f); acc.z = fmaxf(acc.z, 0.f); acc.w = fmaxf(acc.w, 0.f);
        } else if (act == PCL_ACT_SIGMOID) {
            acc.x = sigmoid_fast(acc.x); acc.y = sigmoid_fast(acc.y);
            acc.z = sigmoid_fast(acc.z); acc.w = sigmoid_fast(acc.w);
        }
        out[i] = acc;
    }
}

int launch_reduce_splits_bias_act(const float* partial, float* out, const float* bias, int act, size_t rows, int K,
                                  int splits, cudaStream_t st) {
    if (K % 4 != 0) return PCL_ERR_UNSUPPORTED_SHAPE;
    const size_t n4 = rows * (K / 4);
    if (n4 == 0) return PCL_OK;
    {
        LaunchScope scope(KID_REDUCE_SPLITS, 16.0 * double(n4) * (splits + 1), st);
        reduce_splits_bias_act_kernel<<<grid_for(n4, 256), 256, 0, st>>>(reinterpret_cast<const float4*>(partial),
                                                                          reinterpret_cast<float4*>(out), bias, act, n4, K / 4,
                                                                          splits);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_reduce_splits(const float* partial, float* out, size_t n, int splits, cudaStream_t st) {
    if (n == 0) return PCL_OK;
    {
        LaunchScope scope(KID_REDUCE_SPLITS, 4.0 * double(n) * (splits + 1), st);
        reduce_splits_kernel<<<grid_for(n, 256), 256, 0, st>>>(partial, out, n, splits);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_reduce_splits_sgd(const float* partial, float* w, size_t n, int splits, float lr, cudaStream_t st) {
    if (n == 0) return PCL_OK;
    {
        LaunchScope scope(KID_REDUCE_SPLITS, 4.0 * double(n) * (splits + 2), st);
        reduce_splits_sgd_kernel<<<grid_for(n, 256), 256, 0, st>>>(partial, w, n, splits, lr);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_transpose_flip(const float* w, float* wt_t, int K, int R, int S, int C, cudaStream_t st) {
    if (R * S > 65535) return PCL_ERR_UNSUPPORTED_SHAPE;
    dim3 grid((C + 31) / 32, (K + 31) / 32, R * S);
    if (grid.y > 65535) return PCL_ERR_UNSUPPORTED_SHAPE;
    {
        LaunchScope scope(KID_TRANSPOSE_FLIP, 8.0 * double(K) * R * S * C, st);
        transpose_flip_kernel<<<grid, 256, 0, st>>>(w, wt_t, K, R * S, C);
    }
    return PCL_CHECK_LAUNCH();
}

// Phase-packed backward-data of strided layers with few input maps (see conv_bwd_data_packed in pcl_api.cu).
// wpk[col][i'][j'][k], col = (a*sw + b)*C + c: w[k][a + sh*(Rm-1-i')][b + sw*(Sm-1-j')][c] where that tap exists, else 0;
// columns >= sh*sw*C (padding to a multiple of 4) are zero.
__global__ void __launch_bounds__(256) phase_pack_weights_kernel(const float* __restrict__ w, float* __restrict__ wpk, int K,
                                                                 int R, int S, int C, int sh, int sw, int Rm, int Sm,
                                                                 int cols4) {
    const size_t total = size_t(cols4) * Rm * Sm * K;
    const size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t o = size_t(blockIdx.x) * blockDim.x + threadIdx.x; o < total; o += stride) {
        const int k = int(o % K); size_t t = o / K;
        const int jj = int(t % Sm); t /= Sm;
        const int ii = int(t % Rm); const int col = int(t / Rm);
        float v = 0.f;
        if (col < sh * sw * C) {
            const int c = col % C, ab = col / C, b = ab % sw, a = ab / sw;
            const int r = a + sh * (Rm - 1 - ii), s2 = b + sw * (Sm - 1 - jj);
            if (r < R && s2 < S) v = w[((size_t(k) * R + r) * S + s2) * C + c];
        }
        wpk[o] = v;
    }
}
// dx[n][h][w][c] = t[n][u][v][(a*sw + b)*C + c] with h + pad_h = u*sh + a, w + pad_w = v*sw + b (zeroed where mask <= 0).
// One block per image row of dx: the row's (u, a) are block constants and the per-element index arithmetic is 32-bit.
__global__ void __launch_bounds__(256) phase_unpack_kernel(const float* __restrict__ t, const float* __restrict__ mask,
                                                           float* __restrict__ dx, int H, int W, int C, int sh, int sw,
                                                           int pad_h, int pad_w, int U, int V, int cols4) {
    const size_t row = blockIdx.x;                       // n * H + h
    const size_t n = row / H;
    const int hh = int(row - n * H);
    const int u = (hh + pad_h) / sh, a = (hh + pad_h) - u * sh;
    const float* trow = t + ((n * U + u) * V) * size_t(cols4) + a * sw * C;
    const size_t o0 = row * size_t(W) * C;
    const int row_elems = W * C;
    for (int e = threadIdx.x; e < row_elems; e += blockDim.x) {
        const int ww = e / C, c = e - ww * C;
        const int v = (ww + pad_w) / sw, b = (ww + pad_w) - v * sw;
        float val = __ldg(trow + v * cols4 + b * C + c);
        if (mask && !(__ldg(mask + o0 + e) > 0.f)) val = 0.f;
        dx[o0 + e] = val;
    }
}

int launch_phase_pack_weights(const float* w, float* wpk, int K, int R, int S, int C, int sh, int sw, int Rm, int Sm,
                              int cols4, cudaStream_t st) {
    const size_t total = size_t(cols4) * Rm * Sm * K;
    {
        LaunchScope scope(KID_TRANSPOSE_FLIP, 8.0 * double(total), st);
        phase_pack_weights_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, wpk, K, R, S, C, sh, sw, Rm, Sm, cols4);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_phase_unpack(const float* t, const float* mask, float* dx, int N, int H, int W, int C, int sh, int sw, int pad_h,
                        int pad_w, int U, int V, int cols4, cudaStream_t st) {
    const size_t total = size_t(N) * H * W * C;
    {
        LaunchScope scope(KID_UNPAD_REDUCE, (mask ? 12.0 : 8.0) * double(total), st);
        const size_t rows = size_t(N) * H;
        if (rows > 0x7fffffffu) return PCL_ERR_UNSUPPORTED_SHAPE;
        phase_unpack_kernel<<<unsigned(rows), 256, 0, st>>>(t, mask, dx, H, W, C, sh, sw, pad_h, pad_w, U, V, cols4);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_phase_weights(const float* w, float* wt_t, int K, int R, int S, int C, int a, int b, int stride_h,
                         int stride_w, int Ra, int Sb, cudaStream_t st) {
    const size_t total = size_t(C) * Ra * Sb * K;
    if (total == 0) return PCL_OK;
    {
        LaunchScope scope(KID_TRANSPOSE_FLIP, 8.0 * double(total), st);
        phase_weights_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, wt_t, K, R, S, C, a, b, stride_h, stride_w, Ra, Sb);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_stage_pad_c4(const float* x, float* xs, int N, int H, int W, int C, int pad_h, int pad_w, int slack_pixels,
                        cudaStream_t st) {
    if (slack_pixels < 0 || slack_pixels > 256) return PCL_ERR_UNSUPPORTED_SHAPE;
    const size_t total = size_t(N) * (H + 2 * pad_h) * (W + 2 * pad_w) + slack_pixels;
    {
        LaunchScope scope(KID_STAGE_PAD_C4, 4.0 * double(N) * H * W * C + 16.0 * double(total), st);
        const size_t rows = size_t(N) * (H + 2 * pad_h) + 1;        // + the block that writes the trailing zero pixels
        if (rows > 0x7fffffffu) return PCL_ERR_UNSUPPORTED_SHAPE;
        stage_pad_c4_kernel<<<unsigned(rows), 256, 0, st>>>(x, reinterpret_cast<float4*>(xs), N, H, W, C, pad_h, pad_w,
                                                            slack_pixels);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_stage_w4(const float* w, float* w32, size_t rows, int S, int C, int row_floats, cudaStream_t st) {
    {
        LaunchScope scope(KID_STAGE_W4, double(rows) * (4.0 * S * C + 4.0 * row_floats), st);
        stage_w4_kernel<<<grid_for(rows * row_floats, 256), 256, 0, st>>>(w, w32, rows, S, C, row_floats);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_unpad_reduce(const float* dw4, float* dw, size_t rows, int S, int C, int row_floats, int splits,
                        size_t split_stride, cudaStream_t st) {
    {
        LaunchScope scope(KID_UNPAD_REDUCE, 4.0 * double(rows) * S * C * (splits + 1), st);
        unpad_reduce_kernel<<<grid_for(rows * S * C, 256), 256, 0, st>>>(dw4, dw, rows, S, C, row_floats, splits,
                                                                          split_stride);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_act_grad(float* dy, const float* y, size_t n, int act, cudaStream_t st) {
    if (n == 0 || act == PCL_ACT_NONE) return PCL_OK;
    {
        LaunchScope scope(KID_ACT_GRAD, 12.0 * double(n), st);
        act_grad_kernel<<<grid_for(n, 256), 256, 0, st>>>(dy, y, n, act);
    }
    return PCL_CHECK_LAUNCH();
}

static size_t colsum_rows_per_split(size_t rows) {
    size_t per = (rows + 1183) / 1184;
    if (per < size_t(kColsumMinRows)) per = kColsumMinRows;
    return per;
}
int colsum_splits(size_t rows) {
    const size_t per = colsum_rows_per_split(rows);
    return int((rows + per - 1) / per);
}

// Column groups per block: whole 256-group strips where there are many rows (each row is then read as one contiguous
// run); narrower strips, i.e. more blocks with more rows in flight per block, where a few rows would leave the sum to a
// handful of blocks reading them one after another (the 32 rows of per-tile sums of an FC layer: 9 -> 3 us).
static int colsum_strip(int kv, size_t rows, int splits) {
    int strip = kv < 256 ? kv : 256;
    const size_t rows_in_split = (rows + splits - 1) / splits;
    while (strip > 8 && strip % 2 == 0 && long((kv + strip - 1) / strip) * splits < 64 && size_t(256 / (strip / 2)) <= rows_in_split)
        strip /= 2;
    return strip;
}

int launch_colsum(const float* m, size_t rows, int K, float* partial, float* out, cudaStream_t st) {
    const int splits = colsum_splits(rows);
    const size_t per = colsum_rows_per_split(rows);
    if (splits > 65535) return PCL_ERR_UNSUPPORTED_SHAPE;
    {
        LaunchScope scope(KID_COLSUM, 4.0 * double(rows) * K, st);
        if (K % 4 == 0 && (reinterpret_cast<uintptr_t>(m) & 15) == 0) {
            const int kv = K / 4, strip = colsum_strip(kv, rows, splits);
            colsum_kernel<4><<<dim3((kv + strip - 1) / strip, splits), 256, 0, st>>>(m, rows, K,
                                                                                     splits == 1 ? out : partial, per, strip);
        } else {
            const int strip = colsum_strip(K, rows, splits);
            colsum_kernel<1><<<dim3((K + strip - 1) / strip, splits), 256, 0, st>>>(m, rows, K,
                                                                                    splits == 1 ? out : partial, per, strip);
        }
    }
    if (cudaGetLastError() != cudaSuccess) return PCL_ERR_CUDA;
    if (splits > 1) return launch_reduce_splits(partial, out, size_t(K), splits, st);
    return PCL_OK;
}

int launch_maxpool_fwd(int N, int H, int W, int C, const float* x, float* y, cudaStream_t st, unsigned char* idx) {
    const size_t outs = size_t(N) * (H / 2) * (W / 2);
    {
        LaunchScope scope(KID_MAXPOOL_FWD, 20.0 * double(outs) * C, st);
        if (C % 4 == 0)
            maxpool_fwd_kernel<4><<<grid_for(outs * (C / 4), 256), 256, 0, st>>>(x, y, N, H, W, C, idx);
        else
            maxpool_fwd_kernel<1><<<grid_for(outs * C, 256), 256, 0, st>>>(x, y, N, H, W, C, idx);
    }
    return PCL_CHECK_LAUNCH();
}

// colsum_rows: null, or [maxpool_bwd_colsum_rows()][C] (then C % 4 == 0 and C/4 divides 256)
int launch_maxpool_bwd_idx(int N, int H, int W, int C, const unsigned char* idx, const float* dy, int relu, float* dx,
                           float* colsum_rows, cudaStream_t st) {
    const size_t outs = size_t(N) * (H / 2) * (W / 2);
    if (colsum_rows && maxpool_bwd_colsum_rows(N, H, W, C) == 0) return PCL_ERR_UNSUPPORTED_SHAPE;
    {
        // per output: 1 code byte + 1 dy read + 4 dx written
        LaunchScope scope(KID_MAXPOOL_BWD, 21.0 * double(outs) * C, st);
        if (C % 4 == 0)
            maxpool_bwd_idx_kernel<4><<<grid_for(outs * (C / 4), 256, 16), 256, 0, st>>>(idx, dy, relu, dx, N, H, W, C,
                                                                                          colsum_rows);
        else
            maxpool_bwd_idx_kernel<1><<<grid_for(outs * C, 256), 256, 0, st>>>(idx, dy, relu, dx, N, H, W, C);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_maxpool_bwd(int N, int H, int W, int C, const float* x, const float* dy, const float* mask, float* dx,
                       cudaStream_t st) {
    const size_t outs = size_t(N) * (H / 2) * (W / 2);
    {
        // per output: 4 x read + 1 dy read + 4 dx written (the mask source is x itself in the step)
        LaunchScope scope(KID_MAXPOOL_BWD, 36.0 * double(outs) * C, st);
        if (C % 4 == 0)
            maxpool_bwd_kernel<4><<<grid_for(outs * (C / 4), 256, 16), 256, 0, st>>>(x, dy, mask, dx, N, H, W, C);
        else
            maxpool_bwd_kernel<1><<<grid_for(outs * C, 256), 256, 0, st>>>(x, dy, mask, dx, N, H, W, C);
    }
    return PCL_CHECK_LAUNCH();
}

long maxpool_bwd_colsum_rows(int N, int H, int W, int C) {
    if (C % 4 != 0 || 256 % (C / 4) != 0) return 0;
    const size_t outs = size_t(N) * (H / 2) * (W / 2);
    return grid_for(outs * (C / 4), 256, 16);
}

int launch_maxpool_bwd_colsum(int N, int H, int W, int C, const float* x, const float* dy, const float* mask,
                              float* dx, float* colsum_rows, cudaStream_t st) {
    if (maxpool_bwd_colsum_rows(N, H, W, C) == 0) return PCL_ERR_UNSUPPORTED_SHAPE;
    const size_t outs = size_t(N) * (H / 2) * (W / 2);
    {
        LaunchScope scope(KID_MAXPOOL_BWD, 36.0 * double(outs) * C, st);
        maxpool_bwd_kernel<4><<<grid_for(outs * (C / 4), 256, 16), 256, 0, st>>>(x, dy, mask, dx, N, H, W, C,
                                                                                  colsum_rows);
    }
    return PCL_CHECK_LAUNCH();
}

int launch_softmax_xent(int N, int K, const float* logits, const int* labels, float* loss, float* dlogits,
                        cudaStream_t st) {
    int rc = launch_zero(loss, 1, st);
    if (rc != PCL_OK) return rc;
    {
        LaunchScope scope(KID_SOFTMAX_XENT, 8.0 * double(N) * K, st);
        unsigned int* status = device_status_ptr();
        if (!status) return PCL_ERR_CUDA;
        const int grid = N < 8 * device_sm_count() ? N : 8 * device_sm_count();
        const bool vec = K % 4 == 0 && ((reinterpret_cast<uintptr_t>(logits) | reinterpret_cast<uintptr_t>(dlogits)) & 15) == 0;
        if (K <= 256 * 8 && vec) softmax_xent_regs_kernel<8, 4><<<grid, 256, 0, st>>>(logits, labels, loss, dlogits, N, K, status);
        else if (K <= 256 * 8) softmax_xent_regs_kernel<8, 1><<<grid, 256, 0, st>>>(logits, labels, loss, dlogits, N, K, status);
        else if (K <= 256 * 32 && vec) softmax_xent_regs_kernel<32, 4><<<grid, 256, 0, st>>>(logits, labels, loss, dlogits, N, K, status);
        else if (K <= 256 * 32) softmax_xent_regs_kernel<32, 1><<<grid, 256, 0, st>>>(logits, labels, loss, dlogits, N, K, status);
        else softmax_xent_kernel<<<grid, 256, 0, st>>>(logits, labels, loss, dlogits, N, K, status);
    }
    return PCL_CHECK_LAUNCH();
}

}  // namespace pcl
