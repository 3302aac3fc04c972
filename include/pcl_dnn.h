/*
 * pcl_dnn.h -- C ABI of the B200 (sm_100a) compute library for the training
 * hot path of synchronous SGD: convolution forward / backward-data /
 * weight-gradient, the fully-connected GEMMs, and the SGD weight update,
 * over a whole minibatch.
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 *  - All tensor pointers are DEVICE pointers to fp32 data, contiguous, and at
 *    least 16-byte aligned.  The caller owns every buffer, including the
 *    workspace; the library allocates no device memory.
 *  - Layouts: activations and their gradients are NHWC (N minibatch, H x W
 *    feature map, C feature maps innermost); convolution weights and their
 *    gradients are KRSC (K output maps, R x S kernel, C input maps innermost);
 *    fully-connected weights are [K][C]; outputs of a convolution are NPQK
 *    with P = floor((H + 2*pad_h - R)/stride_h) + 1 (same for Q).
 *  - Outputs are overwritten, never accumulated into.
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *    Every call only enqueues work on that stream and returns; none
 *    synchronises except pcl_last_device_status().
 *  - Return value: PCL_OK or an error code; nothing throws or aborts.  On any
 *    error other than PCL_ERR_DEVICE_TIMEOUT no kernel has been launched.
 *  - Arithmetic: contractions multiply in TF32 (fp32 operands, 10-bit mantissa
 *    inside the tensor core, or full fp32 on the generic kernels) and
 *    accumulate in fp32; elementwise work is fp32.
 *  - Device-side waits are bounded.  A wait that runs out makes the kernel set
 *    a device status word and return early (outputs then undefined);
 *    pcl_last_device_status() reports it as PCL_ERR_DEVICE_TIMEOUT.
 */
#ifndef PCL_DNN_H
#define PCL_DNN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Layer parameters of a 2-D convolution: minibatch, input feature maps,
 * output feature maps, input height/width, kernel height/width, strides and
 * zero padding (the parameters of Algorithm 1, with the printed "- 1" offset
 * generalised to "- pad"). */
typedef struct {
    int N, C, K, H, W, R, S, stride_h, stride_w, pad_h, pad_w;
} pcl_conv_desc;

enum { PCL_ACT_NONE = 0, PCL_ACT_RELU = 1, PCL_ACT_SIGMOID = 2 };

enum {
    PCL_OK = 0,
    PCL_ERR_BAD_ARG = 1,           /* null pointer, non-positive size, unknown enum   */
    PCL_ERR_UNSUPPORTED_SHAPE = 2, /* shape outside what the kernels cover            */
    PCL_ERR_MISALIGNED = 3,        /* a pointer is not 16-byte aligned                */
    PCL_ERR_WORKSPACE = 4,         /* workspace smaller than pcl_*_workspace_bytes()  */
    PCL_ERR_CUDA = 5,              /* a CUDA runtime/driver call failed               */
    PCL_ERR_DEVICE_TIMEOUT = 6,    /* a bounded device-side wait ran out              */
    PCL_ERR_SCRATCH_LIMIT = 7,     /* problem larger than the built-in scratch array  */
    PCL_ERR_BAD_LABEL = 8          /* pcl_softmax_xent met a label outside [0, K)     */
};

enum { PCL_PASS_FWD = 0, PCL_PASS_BWD_DATA = 1, PCL_PASS_BWD_WEIGHTS = 2 };

/* Which kernel family the conv / fc calls use.  PCL_PATH_AUTO picks the tensor
 * core (tcgen05 TF32) kernels whenever the shape is eligible and the generic
 * CUDA-core kernels otherwise; the other two values force one family (a forced
 * tensor-core path returns PCL_ERR_UNSUPPORTED_SHAPE on ineligible shapes).
 * Process-wide setting, intended for tests. */
enum { PCL_PATH_AUTO = 0, PCL_PATH_TENSOR = 1, PCL_PATH_GENERIC = 2 };
int pcl_set_path(int path);

/* Test and tuning knobs (the paper has no counterpart).  Every choice the launchers make -- tiling,
 * tile width, k-steps per pipeline slot, CTA pairs, issuing threads, epilogue form, reduction splits --
 * has a named knob with which the tests pin each kernel variant and the alternatives were measured:
 * TILING (0 plain, 1-3 haloed layouts), BN, KS, KS_HALO, KS_WGRAD, PAIR, PAIR_HALO, PAIR_WGRAD, GRP,
 * ISSUERS, SPLIT_ACC, PIX_WGRAD, XHALO_WGRAD, TMA_STORE, WEIGHTS_IN_PLACE, EPI_WARPS, FC_DW_FORWARD,
 * KSPLIT, RESIDENT_B, KSLICES, SELECT, PACKED_BWD, PLAN_CACHE, WAIT_LIMIT_US (limit of the bounded device-side waits in microseconds,
 * default 2 s; applies to the current device), FAULT_INJECT (test only: 1 / 2 make the next forward-type /
 * weight-gradient launch that runs as single CTAs arm its first pipeline slot for 16 bytes more than it copies,
 * so that the waits on that slot run out, the kernel gives up and returns, and pcl_last_device_status()
 * reports PCL_ERR_DEVICE_TIMEOUT; nothing faults and the context stays usable).  value INT_MIN unsets a knob; pcl_reset_tuning() unsets all.
 * Unset knobs take the launchers' own rules.  Process-wide; nothing is ever read from the environment.
 * Returns PCL_ERR_BAD_ARG for an unknown name. */
int pcl_set_tuning(const char* name, int value);
int pcl_reset_tuning(void);

/* Blocking search (Sec. 2.2-2.3 re-posed: the paper picks its blocks by minimising bytes per flop with a brute-force
 * search; here candidates -- plain or haloed tiling, tile width, single CTAs or CTA pairs -- are scored by a cost
 * model of the tensor pipe, the shared-memory fill rate, the issuing thread and the epilogue warps).  Writes a
 * one-line description of the tiling the forward (PCL_PASS_FWD) or backward-data pass of this layer would launch
 * with under the current knobs, the model's predicted cycles for it and the model's own choice.  Launches
 * nothing.  The SELECT knob = 1 makes the launchers take the model's choice instead of their measured rules. */
int pcl_conv_plan_describe(const pcl_conv_desc* d, int pass, char* buf, size_t buf_bytes);

/* Output spatial size of a convolution.  Returns PCL_ERR_BAD_ARG if the
 * kernel does not fit in the padded input. */
int pcl_conv_out_dims(const pcl_conv_desc* d, int* P, int* Q);

/* Bytes of workspace the given pass needs (0 is possible).  The workspace
 * pointer handed to the pass must be 256-byte aligned. */
size_t pcl_conv_workspace_bytes(const pcl_conv_desc* d, int pass);
size_t pcl_fc_workspace_bytes(int N, int C, int K, int pass);

/* Forward propagation (Algorithm 1):
 *   y[n,p,q,k] = act(bias[k] + sum_{c,r,s} x[n, p*stride_h + r - pad_h,
 *                                            q*stride_w + s - pad_w, c] * w[k,r,s,c])
 * with zero contribution outside the image (cross-correlation, no kernel
 * flip).  x: NHWC in, w: KRSC in, bias: [K] in or NULL, y: NPQK out.
 * act: PCL_ACT_NONE, PCL_ACT_RELU or PCL_ACT_SIGMOID (fused into the epilogue). */
int pcl_conv_fwd(const pcl_conv_desc* d, const float* x, const float* w, const float* bias,
                 float* y, int act, void* ws, size_t ws_bytes, void* cuda_stream);

/* Forward propagation followed by the 2x2 / stride-2 max pooling that the conv -> ReLU -> pool
 * blocks of the VGG-A topology (Sec. 5) apply to it:
 *   y as pcl_conv_fwd();   y_pool[n,p,q,k] = max_{i,j in {0,1}} y[n, 2p+i, 2q+j, k].
 * On the tensor-core path the maxima are taken in the epilogue while the tile is on chip (max
 * commutes with adding the bias and with a monotone activation), which saves re-reading y;
 * other shapes run the pooling kernel after the convolution.  out_h and out_w must be even
 * (PCL_ERR_UNSUPPORTED_SHAPE otherwise).  y_pool: [N][out_h/2][out_w/2][K] out, 16-byte aligned.
 * pool_codes: NULL, or [N][out_h/2][out_w/2][K] bytes out (16-byte aligned): per pooled element the
 * position code of its window, bits 0-1 = position of the first maximum in row-major window order
 * (0: 2p,2q  1: 2p,2q+1  2: 2p+1,2q  3: 2p+1,2q+1), bit 2 set where that maximum is <= 0.  With the
 * codes, pcl_maxpool2x2_bwd_codes() routes the gradient without reading y again.
 * y may be NULL where pcl_conv_fwd_pool_is_fused(d) != 0: the full-resolution output is then not
 * stored at all (a training step that holds y_pool and the codes never reads it again: the pooled
 * layer's backward passes take their ReLU mask from bit 2 of the codes); y_pool and pool_codes are
 * bit-for-bit what the call with y writes.  Elsewhere a NULL y returns PCL_ERR_UNSUPPORTED_SHAPE.
 * Workspace as pcl_conv_fwd(). */
int pcl_conv_fwd_pool_is_fused(const pcl_conv_desc* d);
int pcl_conv_fwd_pool(const pcl_conv_desc* d, const float* x, const float* w, const float* bias,
                      float* y, float* y_pool, unsigned char* pool_codes, int act,
                      void* ws, size_t ws_bytes, void* cuda_stream);

/* Backpropagation (the "Backpropagation" update rule of Sec. 2.1, gather form):
 *   dx[n,h,w,c] = sum over (k,r,s) such that p = (h + pad_h - r)/stride_h and
 *                 q = (w + pad_w - s)/stride_w are integers inside the output
 *                 of dy[n,p,q,k] * w[k,r,s,c]
 * dy: NPQK in, w: KRSC in, dx: NHWC out (every element written; positions no
 * tap reaches get 0).  relu_mask_src: NULL, or an NHWC tensor of dx's shape
 * (the layer's input, i.e. a ReLU output): dx is zeroed where it is <= 0.
 * Workspace: pcl_conv_workspace_bytes(d, PCL_PASS_BWD_DATA) (room for a flipped,
 * transposed copy of w, the "transpose-weights" of Sec. 2.3, plus optional room for
 * a split reduction; the tensor-core path reads w in place instead when C is a
 * multiple of 32, and a smaller or absent workspace then only forgoes the split). */
int pcl_conv_bwd_data(const pcl_conv_desc* d, const float* dy, const float* w,
                      const float* relu_mask_src, float* dx,
                      void* ws, size_t ws_bytes, void* cuda_stream);

/* Backpropagation that also returns the per-map sums of what it wrote:
 *   dx as pcl_conv_bwd_data();  dx_colsum[c] = sum_{n,h,w} dx[n,h,w,c]   (after the mask).
 * With the ReLU mask fused, dx is the gradient w.r.t. the pre-activation of the
 * layer below, so dx_colsum is that layer's bias gradient: the sums are formed
 * in the epilogue while the tile is on chip instead of re-reading dx from
 * memory.  Deterministic (fixed summation order).  dx_colsum: [C] out.
 * Workspace: pcl_conv_bwd_data_colsum_workspace_bytes(d). */
size_t pcl_conv_bwd_data_colsum_workspace_bytes(const pcl_conv_desc* d);
int pcl_conv_bwd_data_colsum(const pcl_conv_desc* d, const float* dy, const float* w,
                             const float* relu_mask_src, float* dx, float* dx_colsum,
                             void* ws, size_t ws_bytes, void* cuda_stream);

/* Weight-gradient update (Sec. 2.1):
 *   dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride_h + r - pad_h, q*stride_w + s - pad_w, c]
 *   dbias[k]    = sum_{n,p,q} dy[n,p,q,k]                  (if dbias != NULL)
 * x: NHWC in, dy: NPQK in, dw: KRSC out, dbias: [K] out or NULL.
 * The minibatch/pixel reduction is split across thread blocks ("privatise and
 * reduce", Sec. 2.5).  deterministic != 0: partial sums go to the workspace and
 * a second pass adds them in a fixed order (bitwise reproducible);
 * deterministic == 0: partial sums are added with fp32 atomics (order varies). */
int pcl_conv_bwd_weights(const pcl_conv_desc* d, const float* x, const float* dy,
                         float* dw, float* dbias, int deterministic,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Weight-gradient update with the SGD step applied by its own second pass (Sec. 3.1: a layer's new weights are
 * only needed before its next forward pass, so the update need not wait for a pass of its own):
 *   w[k,r,s,c] <- w[k,r,s,c] - lr * dw[k,r,s,c],   dw as in pcl_conv_bwd_weights(), never written to memory where the
 * reduction over pixels is split (its second pass adds the partial sums in the fixed order and applies the update);
 * otherwise dw goes to the workspace and the update follows.  Bit-identical to pcl_conv_bwd_weights() (deterministic)
 * followed by pcl_sgd_update().  The caller must have issued every reader of the OLD weights (the layer's
 * backpropagation) before this call.  w: KRSC in/out (device, 16-byte aligned); dbias: [K] out or NULL, as above.
 * Workspace: pcl_conv_bwd_weights_sgd_workspace_bytes(d), 256-byte aligned.  Errors as pcl_conv_bwd_weights(). */
size_t pcl_conv_bwd_weights_sgd_workspace_bytes(const pcl_conv_desc* d);
int pcl_conv_bwd_weights_sgd(const pcl_conv_desc* d, const float* x, const float* dy, float* w, float lr,
                             float* dbias, void* ws, size_t ws_bytes, void* cuda_stream);

/* Weight-gradient update of a layer whose output went through the 2x2 / stride-2 max pool (the
 * conv -> ReLU -> pool blocks of the VGG-A topology, Sec. 5), taken straight from the POOLED gradient:
 *   dy[n,p,q,k] = dy_pool[n,p/2,q/2,k]  where (p%2)*2 + q%2 == pool_codes[n,p/2,q/2,k] & 3
 *                                       (and, if relu_mask != 0, bit 2 of that code is clear), else 0;
 *   dw, dbias as pcl_conv_bwd_weights() of that dy (two-pass, bitwise reproducible).
 * I.e. pcl_maxpool2x2_bwd_codes() followed by pcl_conv_bwd_weights(), but dy is never written to or
 * read from memory: the kernel builds its dy tiles on chip.  For a layer with no backward-data pass of
 * its own (the first layer: Sec. 3.1 skips its backpropagation) nothing else needs dy.
 * dy_pool: [N][out_h/2][out_w/2][K] in, pool_codes: same shape, bytes, in (codes as written by
 * pcl_conv_fwd_pool / pcl_maxpool2x2_fwd_codes), both 16-byte aligned; dbias: [K] out or NULL.
 * Available where pcl_conv_bwd_weights_pooled_is_fused(d) != 0 (the few-channel first-layer path, even
 * out_h and out_w, K % 4 == 0); elsewhere PCL_ERR_UNSUPPORTED_SHAPE (run the two calls instead).
 * Workspace: pcl_conv_bwd_weights_pooled_workspace_bytes(d), 256-byte aligned. */
int pcl_conv_bwd_weights_pooled_is_fused(const pcl_conv_desc* d);
size_t pcl_conv_bwd_weights_pooled_workspace_bytes(const pcl_conv_desc* d);
int pcl_conv_bwd_weights_pooled(const pcl_conv_desc* d, const float* x, const float* dy_pool,
                                const unsigned char* pool_codes, int relu_mask, float* dw, float* dbias,
                                void* ws, size_t ws_bytes, void* cuda_stream);

/* The same from the staged input the layer's forward call left behind (the paper has no counterpart).  On the
 * few-channel path pcl_conv_fwd() / pcl_conv_fwd_pool() first write a 4-channel, halo-padded, TF32-rounded copy of x
 * to the first pcl_conv_staged_input_bytes(d) bytes of their workspace; a caller that keeps that workspace untouched
 * until the backward pass hands its address to this call as x_staged (256-byte aligned) and saves staging x a second
 * time.  Same result as pcl_conv_bwd_weights_pooled(), bit for bit.  pcl_conv_staged_input_bytes() is 0 for layers
 * that stage nothing. */
size_t pcl_conv_staged_input_bytes(const pcl_conv_desc* d);
int pcl_conv_bwd_weights_pooled_staged(const pcl_conv_desc* d, const float* x_staged, const float* dy_pool,
                                       const unsigned char* pool_codes, int relu_mask, float* dw, float* dbias,
                                       void* ws, size_t ws_bytes, void* cuda_stream);

/* Fully-connected forward: the k_h = k_w = out_h = out_w = 1 case of Algorithm 1
 * (Sec. 2.1):  y[n,k] = act(bias[k] + sum_c x[n,c] * w[k,c]).
 * x: [N][C], w: [K][C], bias: [K] or NULL, y: [N][K].
 * act: NONE, RELU or SIGMOID.
 * Workspace: optional.  With pcl_fc_workspace_bytes(N, C, K, PCL_PASS_FWD) bytes (256-byte aligned) a
 * layer with few output tiles and a long reduction splits the reduction over more CTAs and adds the
 * partial results in a fixed order in a second pass; without it the same result is computed unsplit
 * (up to the order of the fp32 additions).  pcl_conv_fwd() takes the same optional scratch
 * (pcl_conv_workspace_bytes(d, PCL_PASS_FWD)). */
int pcl_fc_fwd(int N, int C, int K, const float* x, const float* w, const float* bias,
               float* y, int act, void* ws, size_t ws_bytes, void* cuda_stream);

/* Fully-connected backward (same special case of the two update rules):
 *   dz = dy * act'(y)   (ReLU: [y > 0]; sigmoid: y(1-y); written back into dy)
 *   dx[n,c] = sum_k dz[n,k] * w[k,c]      (skipped if dx == NULL: first layer)
 *   dw[k,c] = sum_n dz[n,k] * x[n,c]
 *   dbias[k] = sum_n dz[n,k]              (skipped if dbias == NULL)
 * y is only read when act != NONE (may be NULL otherwise).  Workspace size:
 * pcl_fc_workspace_bytes(N, C, K, PCL_PASS_BWD_DATA). */
int pcl_fc_bwd(int N, int C, int K, const float* x, const float* w, const float* y, int act,
               float* dy, float* dx, float* dw, float* dbias,
               void* ws, size_t ws_bytes, void* cuda_stream);

/* pcl_fc_bwd() with the layer below's share of the work folded into the backpropagation kernel's epilogue
 * (the paper has no counterpart; same update rules, Sec. 2.1):
 *   dx[n,c]      = (sum_k dz[n,k] * w[k,c]) * x_act'(x[n,c])   x_act = the activation that produced x (NONE, RELU:
 *                  [x > 0], SIGMOID: x(1-x)): dx is then the gradient w.r.t. the pre-activation of the layer
 *                  below, i.e. the dz that layer's own call would otherwise form with a pass of its own;
 *   dx_colsum[c] = sum_n dx[n,c]   (NULL to skip): with x_act set, the bias gradient of the layer below.
 * The layer below is then called with act = PCL_ACT_NONE and dbias = NULL.  Deterministic.  Workspace as pcl_fc_bwd(). */
int pcl_fc_bwd_fused(int N, int C, int K, const float* x, const float* w, const float* y, int act,
                     float* dy, float* dx, int x_act, float* dx_colsum, float* dw, float* dbias,
                     void* ws, size_t ws_bytes, void* cuda_stream);

/* pcl_fc_bwd_fused() with the SGD step folded in: dx (and dx_colsum) are computed from the OLD weights first, then
 *   w[k,c] <- w[k,c] - lr * dw[k,c]
 * in place, without dw ever being stored (the weight-gradient GEMM's epilogue reads w and writes the updated value,
 * or the second pass of its split reduction does).  dbias as in pcl_fc_bwd().  Bit-identical to pcl_fc_bwd_fused()
 * followed by pcl_sgd_update() on w.  w: [K][C] in/out.  Workspace: pcl_fc_bwd_fused_sgd_workspace_bytes(N, C, K). */
size_t pcl_fc_bwd_fused_sgd_workspace_bytes(int N, int C, int K);
int pcl_fc_bwd_fused_sgd(int N, int C, int K, const float* x, float* w, const float* y, int act,
                         float* dy, float* dx, int x_act, float* dx_colsum, float lr, float* dbias,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Launch plans.  What a tensor-core launch needs besides its data -- the tiling, the kernel's parameter block, its TMA
 * tensor maps, the grid -- follows from the call's arguments alone, so it is built once per distinct argument set
 * (descriptor, pointers, strides, options; per device; per setting of the tuning knobs) and kept in a host-side
 * cache (a few hundred bytes per plan, at most 512 plans per kernel family, then the cache starts over).  A training
 * step that calls with the same buffers every iteration selects tilings and encodes tensor maps once per layer and
 * pass.  Thread-safe.  The PLAN_CACHE knob (pcl_set_tuning) set to 0 builds every launch's plan afresh.
 * pcl_plan_cache_stats: launches served from the cache / launches that built a plan, since the library was loaded
 * (host counters; either pointer may be NULL). */
int pcl_plan_cache_stats(unsigned long long* hits, unsigned long long* misses);

/* Vanilla SGD (Sec. 1: algorithm and hyper-parameters untouched):
 *   w[i] <- w[i] - lr * dw[i],  i < n.   w, dw only need 4-byte alignment. */
int pcl_sgd_update(float* w, const float* dw, size_t n, float lr, void* cuda_stream);

/* Glue the VGG-A / DNN topologies of Sec. 5 need between the passes above. */
/* 2x2 window, stride 2, no padding; H and W even.  x: NHWC, y: N,H/2,W/2,C. */
int pcl_maxpool2x2_fwd(int N, int H, int W, int C, const float* x, float* y, void* cuda_stream);
/* dx gets dy at the first maximum of each window (row-major window order) and 0
 * elsewhere; then, if relu_mask_src != NULL (NHWC, x's shape), dx is zeroed
 * where relu_mask_src <= 0. */
int pcl_maxpool2x2_bwd(int N, int H, int W, int C, const float* x, const float* dy,
                       const float* relu_mask_src, float* dx, void* cuda_stream);
/* pcl_maxpool2x2_bwd() plus dx_colsum[c] = sum_{n,h,w} dx[n,h,w,c] (the bias gradient of the
 * convolution whose ReLU output was pooled).  Deterministic.  Workspace:
 * pcl_maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C). */
size_t pcl_maxpool2x2_bwd_colsum_workspace_bytes(int N, int H, int W, int C);
int pcl_maxpool2x2_bwd_colsum(int N, int H, int W, int C, const float* x, const float* dy,
                              const float* relu_mask_src, float* dx, float* dx_colsum,
                              void* ws, size_t ws_bytes, void* cuda_stream);
/* Pooling with position codes (see pcl_conv_fwd_pool): the forward pass also writes codes[n,p,q,c];
 * the backward pass takes the codes instead of x:  dx gets dy at the coded position of each window
 * and 0 elsewhere; relu_mask != 0: windows whose code has bit 2 set (maximum <= 0, i.e. the ReLU
 * that produced x was inactive there) get 0 everywhere, which equals pcl_maxpool2x2_bwd() with
 * relu_mask_src = x.  dx_colsum: NULL, or [C] out = sum_{n,h,w} dx[n,h,w,c] (deterministic), then the
 * workspace of pcl_maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C) is needed. */
int pcl_maxpool2x2_fwd_codes(int N, int H, int W, int C, const float* x, float* y, unsigned char* codes,
                             void* cuda_stream);
int pcl_maxpool2x2_bwd_codes(int N, int H, int W, int C, const unsigned char* codes, const float* dy,
                             int relu_mask, float* dx, float* dx_colsum,
                             void* ws, size_t ws_bytes, void* cuda_stream);
/* loss = -(1/N) sum_n log softmax(logits[n,:])[labels[n]]  (device scalar, overwritten)
 * dlogits = (softmax(logits) - onehot(labels)) / N.  labels: device int32 [N].
 * A label outside [0, K) is never used as an index: that row gets no target (its gradient is
 * softmax/N) and no loss term, and the next pcl_last_device_status() returns PCL_ERR_BAD_LABEL.
 * dlogits is bitwise reproducible; the loss scalar is summed over the rows with fp32 atomics, so
 * its last bits may differ from run to run. */
int pcl_softmax_xent(int N, int K, const float* logits, const int* labels,
                     float* loss, float* dlogits, void* cuda_stream);

/* Synchronises the stream, then reads and clears the device status word of the
 * current device.  PCL_OK, PCL_ERR_DEVICE_TIMEOUT, PCL_ERR_BAD_LABEL or PCL_ERR_CUDA. */
int pcl_last_device_status(void* cuda_stream);
/* Which wait gave up when pcl_last_device_status() last returned PCL_ERR_DEVICE_TIMEOUT (0 if it never did):
 * 0x101 producer waiting for a free slot, 0x102 MMA issuer waiting for operands, 0x103 MMA issuer waiting for a
 * free accumulator, 0x104 epilogue waiting for an accumulator, 0x106 MMA issuer waiting for its turn.  Diagnostic. */
unsigned int pcl_last_wait_code(void);

/* Number of kernels this library has launched since it was loaded. */
unsigned long long pcl_launch_count(void);

/* Backward-data for callers that cannot allocate device memory (the paper has
 * no counterpart; this is a convenience of the library).
 *
 * Same result as pcl_conv_bwd_data(), but the caller passes no workspace: the
 * flipped, transposed weight copy goes into a fixed array inside the library's
 * device image.  Meant for code that is handed tensors but has no allocator to
 * ask -- a plugin, a serving loop whose device memory all belongs to someone
 * else's pool, any place where cudaMalloc is off limits.  The call itself makes
 * no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *  - Capacity: pcl_noalloc_scratch_bytes() = 16 MiB.  What has to fit is the
 *    transposed copy, which only layers with C % 32 != 0 need: for those
 *    K*R*S*C <= 4 194 304 weights, else PCL_ERR_SCRATCH_LIMIT and nothing is
 *    launched.  Layers with C % 32 == 0 are read in place and accepted at any size.
 *    (Where the regular call would also use scratch to split a long reduction, this
 *    one splits only as far as the array's remaining room allows: same result up to
 *    the order of the fp32 additions when the split count differs.)
 *    Every GPU that loads the library holds these 16 MiB until the process ends.
 *  - The first call on each device looks up the array's device address (one
 *    runtime query, no allocation); make that first call before any stream
 *    capture begins.
 *  - All calls share the one array.  Each call overwrites it completely before
 *    reading it, so calls issued one after another on a stream are fine; calls
 *    whose kernels may overlap on the GPU (different streams, or different host
 *    threads on different streams) race on it and must be serialised by the
 *    caller.
 * Arguments as for pcl_conv_bwd_data() without ws / ws_bytes. */
int pcl_conv_bwd_data_noalloc(const pcl_conv_desc* d, const float* dy, const float* w,
                              const float* relu_mask_src, float* dx, void* cuda_stream);
size_t pcl_noalloc_scratch_bytes(void);

/* Optional per-kernel timing (the paper has no counterpart; measurement aid).
 * Between pcl_profile_begin() and pcl_profile_end() every kernel launch of the
 * library is bracketed by two CUDA events on its launching stream.
 * pcl_profile_end() waits for those events, stops the bracketing and returns, per
 * kernel family that ran, the number of launches, the summed event time and the
 * summed algorithmic work (flops for the contraction kernels, bytes for the
 * memory-bound ones), separately for each pass the launches belonged to: `name` is
 * "<pass>/<kernel>" with pass one of conv_fwd, conv_bwd_data, conv_bwd_weights, fc_fwd,
 * fc_bwd, other (the ABI call that made the launch).  A contraction launch counts the
 * layer's own 2*N*K*P*Q*C*R*S (Comp of Sec. 3.1 per pass), also where the kernel runs on
 * a zero-padded view of the layer.  stats: HOST array of max_stats entries; *n_stats
 * entries are filled.  Event objects are created on first use and reused. */
typedef struct {
    char name[64];
    unsigned long long launches;
    double total_ms;
    double work;
} pcl_kernel_stat;
int pcl_profile_begin(void);
int pcl_profile_end(pcl_kernel_stat* stats, int max_stats, int* n_stats);

const char* pcl_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* PCL_DNN_H */
