// Ceiling probes: tiny kernels that measure, on the GPU at hand, the on-chip rates that bound
// the 3D-DSA kernels (the operator is a gather / scatter of 256..512-byte rows, not a
// stream): random row gathers served by L2, fp32 vector reductions into L2, and the FMA
// issue rate with and without bf16 operands.  They are measurement aids for the benchmark;
// the paper has no counterpart.  Every probe works on a caller-provided device buffer,
// launches one kernel on the caller's stream and reports how much work that launch does, so
// the caller times it with its own events.
#include <stdint.h>

#include "../../include/dsa3d.h"
#include "dsa3d_common.cuh"

namespace {

__device__ __forceinline__ uint32_t hash32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352dU; x ^= x >> 15; x *= 0x846ca68bU; x ^= x >> 16;
    return x;
}

constexpr int kProbeBlocks = 148 * 8, kProbeThreads = 256;

// Every half-warp reads one random 256-byte row per step with 16-byte loads (the access
// shape of the corner gathers of a 128-channel bf16 head).
__global__ void __launch_bounds__(kProbeThreads)
probe_gather_kernel(const uint4* __restrict__ base, uint32_t nrows, int iters, float* sink) {
    const int lane = threadIdx.x & 31, sub = lane >> 4, gl = lane & 15;
    const uint32_t wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    uint32_t s = wid * 977u + 12345u;
    float acc = 0.0f;
    for (int i = 0; i < iters; i += 8) {
        uint4 r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t row = hash32(s + (i + j) * 2 + sub) % nrows;
            r[j] = __ldg(base + static_cast<size_t>(row) * 16 + gl);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) acc += __uint_as_float(r[j].x) + __uint_as_float(r[j].w);
    }
    if (acc == 123.456f) sink[0] = acc;
}

// Every warp adds 512 bytes (one 128-channel fp32 row) to a random row per step.
__global__ void __launch_bounds__(kProbeThreads)
probe_red_kernel(float* __restrict__ base, uint32_t nrows, int iters) {
    const int lane = threadIdx.x & 31;
    const uint32_t wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t s = wid * 977u + 777u;
    for (int i = 0; i < iters; ++i) {
        const uint32_t row = hash32(s + i) % nrows;
        float* p = base + static_cast<size_t>(row) * 128 + lane * 4;
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(0.f), "f"(0.f), "f"(0.f), "f"(0.f)
                     : "memory");
    }
}

// 64 FMAs per thread and step on register data: kind 0 plain fp32, kind 1 the mixed
// bf16 x bf16 -> fp32 instruction the bf16 kernels use.
__global__ void __launch_bounds__(512)
probe_fma_kernel(int iters, int kind, const uint32_t* __restrict__ seed, float* sink) {
    uint32_t w[4], q[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) { w[k] = seed[(threadIdx.x + k * 32) & 255]; q[k] = seed[(threadIdx.x + 128 + k * 32) & 255]; }
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (kind == 0) {
        float a[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) { a[2 * k] = __uint_as_float(w[k] & 0xffff0000u); a[2 * k + 1] = __uint_as_float(q[k] & 0xffff0000u); }
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] = fmaf(a[k], a[(k + u) & 7], acc[k]);
        }
    } else {
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    unsigned short wl, wh, ql, qh;
                    dsa3d::split_b32(w[k], wl, wh);
                    dsa3d::split_b32(q[(k + u) & 3], ql, qh);
                    acc[2 * k] = dsa3d::fma_bf16(ql, wl, acc[2 * k]);
                    acc[2 * k + 1] = dsa3d::fma_bf16(qh, wh, acc[2 * k + 1]);
                }
            }
            w[i & 3] ^= static_cast<uint32_t>(i) << 16;        // keep the data changing
        }
    }
    float s = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; ++k) s += acc[k];
    if (s == 1.2345f) sink[0] = s;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

int dsa3d_probe_gather(const void* buffer, size_t working_set_bytes, int iters, double* bytes_per_launch,
                       void* stream) {
    if (!buffer || !bytes_per_launch) return DSA3D_ERR_NULL_POINTER;
    if (!aligned16(buffer)) return DSA3D_ERR_MISALIGNED;
    if (working_set_bytes < 256 || working_set_bytes / 256 > 0xffffffffull || iters < 8 || iters % 8) return DSA3D_ERR_BAD_SHAPE;
    const uint32_t nrows = static_cast<uint32_t>(working_set_bytes / 256);
    probe_gather_kernel<<<kProbeBlocks, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(buffer), nrows, iters,
        static_cast<float*>(const_cast<void*>(buffer)));   // the sink write never happens
    *bytes_per_launch = static_cast<double>(kProbeBlocks) * (kProbeThreads / 32) * iters * 512.0;
    return cudaGetLastError() == cudaSuccess ? DSA3D_OK : DSA3D_ERR_CUDA;
}

int dsa3d_probe_red(void* buffer, size_t working_set_bytes, int iters, double* bytes_per_launch, void* stream) {
    if (!buffer || !bytes_per_launch) return DSA3D_ERR_NULL_POINTER;
    if (!aligned16(buffer)) return DSA3D_ERR_MISALIGNED;
    if (working_set_bytes < 512 || working_set_bytes / 512 > 0xffffffffull || iters < 1) return DSA3D_ERR_BAD_SHAPE;
    const uint32_t nrows = static_cast<uint32_t>(working_set_bytes / 512);
    probe_red_kernel<<<kProbeBlocks, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<float*>(buffer), nrows, iters);
    *bytes_per_launch = static_cast<double>(kProbeBlocks) * (kProbeThreads / 32) * iters * 512.0;
    return cudaGetLastError() == cudaSuccess ? DSA3D_OK : DSA3D_ERR_CUDA;
}

int dsa3d_probe_fma(const void* seed_1kb, int iters, int kind, double* fma_per_launch, void* stream) {
    if (!seed_1kb || !fma_per_launch) return DSA3D_ERR_NULL_POINTER;
    if (iters < 1 || (kind != 0 && kind != 1)) return DSA3D_ERR_BAD_SHAPE;
    constexpr int blocks = 148 * 4, threads = 512;
    probe_fma_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        iters, kind, static_cast<const uint32_t*>(seed_1kb),
        static_cast<float*>(const_cast<void*>(seed_1kb)));   // the sink write never happens
    *fma_per_launch = static_cast<double>(blocks) * threads * iters * 64.0;
    return cudaGetLastError() == cudaSuccess ? DSA3D_OK : DSA3D_ERR_CUDA;
}

}  // extern "C"
