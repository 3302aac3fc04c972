/*
 * TEST INFRASTRUCTURE -- the CPU oracle for the convolution / fully-connected
 * training passes.  Plain, slow, fp64.  Only the tests, the smoke check and the
 * benchmark's cpu-baseline leg may load this library; the CUDA product path
 * shares no code with it and never calls it.
 *
 * What it computes is the plain definition of the three passes (Algorithm 1
 * and the two update rules that follow it in Sec. 2.1), evaluated in double
 * precision with a fixed loop order.  OpenMP is used over independent outputs
 * only, so results are bitwise reproducible for any thread count.
 *
 * Build:  gcc -O2 -fopenmp -shared -fPIC -o libpcl_oracle.so pcl_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int N, C, K, H, W, R, S, stride_h, stride_w, pad_h, pad_w;
} conv_shape;

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_SIGMOID = 2 };

/* P = floor((H + 2*pad - R) / stride) + 1 */
static int64_t out_dim(int64_t in, int64_t k, int64_t stride, int64_t pad)
{
    int64_t span = in + 2 * pad - k;
    if (span < 0) return 0;
    return span / stride + 1;
}

static double apply_act(double v, int act)
{
    if (act == ACT_RELU) return v > 0.0 ? v : 0.0;
    if (act == ACT_SIGMOID) return 1.0 / (1.0 + exp(-v));
    return v;
}

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_out_dims(const conv_shape *d, int64_t *P, int64_t *Q)
{
    *P = out_dim(d->H, d->R, d->stride_h, d->pad_h);
    *Q = out_dim(d->W, d->S, d->stride_w, d->pad_w);
}

#define CAT2(a, b) a##b
#define CAT(a, b) CAT2(a, b)

#define IN_T float
#define FN(name) CAT(name, _f32)
#include "conv_loops.inc"
#undef IN_T
#undef FN

#define IN_T double
#define FN(name) CAT(name, _f64)
#include "conv_loops.inc"
#undef IN_T
#undef FN
