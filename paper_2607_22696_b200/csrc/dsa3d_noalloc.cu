// dsa3d_backward_noalloc: the backward pass for callers that cannot obtain device scratch.
//
// Some hosts of this library have no way to hand it a workspace: code that runs inside a
// framework's captured or pre-planned region where every allocation was fixed up front,
// plug-ins whose embedding application owns the only device allocator and exposes no
// scratch API, or real-time loops in which cudaMalloc (which may synchronise the whole
// device) is forbidden.  For them the fp32 dK/dV accumulators live in a fixed array inside
// the library image itself.  Nothing here calls cudaMalloc, cudaFree or any allocating
// routine.
#include <stdint.h>

#include <mutex>

#include "../../include/dsa3d.h"
#include "dsa3d_kernels.h"

namespace {

// 2 x 8 Mi floats = 64 MiB: room for dK and dV accumulators of problems with up to
// DSA3D_NOALLOC_MAX_ELEMENTS = T*H*W*heads*d elements.  The array is part of the module
// image, so every GPU that loads the library keeps these 64 MiB until the process exits.
constexpr size_t kMaxElements = DSA3D_NOALLOC_MAX_ELEMENTS;
static __device__ __align__(256) float g_scratch[2 * kMaxElements];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_scratch_ptr[kMaxDevices] = {};   // device address of g_scratch, per device ordinal

thread_local int g_noalloc_cuda_error = 0;

// `g_scratch` in host code is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, once per device, with that device current.
int scratch_for_current_device(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_noalloc_cuda_error = static_cast<int>(e); return DSA3D_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return DSA3D_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess || !p) {
            g_noalloc_cuda_error = static_cast<int>(e);
            return DSA3D_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_ptr[dev];
    return DSA3D_OK;
}

}  // namespace

extern "C" {

size_t dsa3d_backward_noalloc_max_elements(void) { return kMaxElements; }

int dsa3d_backward_noalloc_last_cuda_error(void) { return g_noalloc_cuda_error; }

int dsa3d_backward_noalloc(const void* q, const void* k, const void* v, const float* offsets,
                           const float* lse, const void* dout, int T, int H, int W, int heads, int d,
                           const int window[3], void* dq, void* dk, void* dv, float* doffsets, int dtype,
                           void* stream) {
    if (!q || !k || !v || !offsets || !lse || !dout || !dq || !dk || !dv || !doffsets || !window)
        return DSA3D_ERR_NULL_POINTER;
    if (T < 1 || H < 1 || W < 1 || heads < 1 || d < 1) return DSA3D_ERR_BAD_SHAPE;
    // Reject anything that does not fit the fixed array before touching the device.
    unsigned long long elements = 1;                // grows factor by factor, so it cannot wrap
    const int factors[5] = {T, H, W, heads, d};
    for (int f : factors) {
        elements *= static_cast<unsigned long long>(f);
        if (elements > kMaxElements) return DSA3D_ERR_WORKSPACE;
    }
    if (dtype == DSA3D_F32)   // fp32 storage accumulates straight into dk / dv: no scratch at all
        return dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv,
                                    doffsets, nullptr, 0, dtype, stream, false);
    float* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != DSA3D_OK) return rc;
    // The shared implementation validates the rest, clears the accumulators (the array keeps
    // whatever the previous call left) and scatters every dK/dV contribution straight into
    // them: the tile pre-reduction of dsa3d_backward needs far more scratch than this array.
    return dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                                scratch, 2 * kMaxElements * sizeof(float), dtype, stream, false);
}

}  // extern "C"
