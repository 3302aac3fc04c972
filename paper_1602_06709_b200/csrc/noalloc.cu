// Backward-data entry point for callers that cannot allocate device memory.
//
// pcl_conv_bwd_data() needs a caller-provided workspace for the flipped,
// transposed copy of the weights.  Some callers have no way to provide one:
// a plugin that is handed tensors but no allocator, a serving loop whose
// process gave all device memory to a pool it does not own, code running where
// cudaMalloc is forbidden.  For them the workspace lives here, in a fixed-size
// array in the library's own device image.  Every GPU that loads the library
// carries these 16 MiB until the process exits, which is why the capacity is
// modest and fixed.
#include <mutex>

#include "pcl_internal.h"

namespace {

// Capacity of the built-in scratch: 4 Mi floats = 16 MiB.  What must fit is the
// transposed copy of the K*R*S*C weights, and only for layers that need one
// (C not a multiple of 32); layers whose weights are read in place need no
// scratch and are accepted at any size.
constexpr size_t kScratchFloats = size_t(4) << 20;

// File-scope device array.  In host code this name is only a handle for the
// runtime: it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

// Device address of the array on the current device, looked up once per device.
float* scratch_address(int* rc) {
    static float* cache[64] = {};
    static std::mutex mu;
    *rc = PCL_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *rc = PCL_ERR_CUDA; return nullptr; }
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch) != cudaSuccess || !ptr) {
            *rc = PCL_ERR_CUDA;
            return nullptr;
        }
        cache[dev] = ptr;
    }
    return cache[dev];
}

}  // namespace

extern "C" int pcl_conv_bwd_data_noalloc(const pcl_conv_desc* d, const float* dy, const float* w,
                                         const float* relu_mask_src, float* dx, void* cuda_stream) {
    if (!d) return PCL_ERR_BAD_ARG;
    int P = 0, Q = 0;
    int rc = pcl_conv_out_dims(d, &P, &Q);
    if (rc != PCL_OK) return rc;
    // Only the transposed weight copy is mandatory.  The regular entry point also uses scratch, when it has some,
    // to split long reductions over more thread blocks; here it splits as far as the rest of the array allows.
    const size_t need = pcl::bwd_data_transposed_bytes(*d);
    if (need > kScratchFloats * sizeof(float)) return PCL_ERR_SCRATCH_LIMIT;
    float* scratch = scratch_address(&rc);
    if (rc != PCL_OK) return rc;
    // The transposed weights (and any split partials) are written in full before they are read, so nothing
    // has to be cleared between calls; what the previous call left in the array is simply overwritten.
    return pcl_conv_bwd_data(d, dy, w, relu_mask_src, dx, scratch, kScratchFloats * sizeof(float), cuda_stream);
}

extern "C" size_t pcl_noalloc_scratch_bytes(void) { return kScratchFloats * sizeof(float); }
