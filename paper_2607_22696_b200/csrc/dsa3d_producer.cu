// The two layers that surround the attention operator in Eq. 1 and feed it its offsets:
//   dwconv3d_kernel        depthwise 3-D convolution on channels-last activations (first term of
//                          Eq. 1; first stage of the offset predictor of the Formulation section)
//   offsets_gemm_kernel    offsets = u . w^T + bias, the linear layer of the offset predictor, as
//                          a dense bf16 contraction on the 5th-generation tensor cores:
//                          TMA tiles (128-byte swizzle) -> tcgen05.mma -> fp32 accumulators in
//                          TMEM -> bias + fp32 stores.  Persistent, one CTA per SM, warp-
//                          specialised (TMA producer, MMA issuer, four epilogue warps), four
//                          shared-memory stages, two TMEM accumulator buffers so the epilogue of
//                          one tile overlaps the contraction of the next.  By default pairs of CTAs
//                          share a 256-row tile (offsets_gemm_pair_kernel, cta_group::2).
//   offsets_linear_f32_kernel  the same layer in plain fp32 FMAs for fp32 storage.
// Every wait on an mbarrier is bounded; a wait that runs out raises a device flag (readable
// with dsa3d_device_timeout_flag) and the roles drain and free TMEM instead of spinning.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <mutex>

#include "../../include/dsa3d.h"
#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace {

using namespace dsa3d;

__device__ int g_timeout_flag = 0;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------------------------------
// Depthwise convolution.  A thread owns 8 consecutive channels (one 16-byte vector of bf16,
// two of fp32) of RX = 8 consecutive outputs along x; per (dt, dy) row of the kernel it loads
// the kw weight vectors and the RX + kw - 1 input vectors once and slides the taps over them
// in registers.  Consecutive threads take consecutive channel vectors (coalesced rows).
// ------------------------------------------------------------------------------------------
constexpr int kConvRX = 8;
constexpr int kConvMaxKw = 7;

template <typename T> struct Vec8;
template <> struct Vec8<__nv_bfloat16> {
    using Raw = uint4;
    static __device__ __forceinline__ Raw load_raw(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
    static __device__ __forceinline__ Raw zero_raw() { return make_uint4(0u, 0u, 0u, 0u); }
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) { widen(load_raw(p), f); }
    static __device__ __forceinline__ void widen(const Raw& r, float (&f)[8]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};
template <> struct Vec8<float> {
    struct Raw { float4 a, b; };
    static __device__ __forceinline__ Raw load_raw(const float* p) {
        Raw r;
        r.a = __ldg(reinterpret_cast<const float4*>(p));
        r.b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        return r;
    }
    static __device__ __forceinline__ Raw zero_raw() {
        Raw r;
        r.a = r.b = make_float4(0.f, 0.f, 0.f, 0.f);
        return r;
    }
    static __device__ __forceinline__ void load(const float* p, float (&f)[8]) { widen(load_raw(p), f); }
    static __device__ __forceinline__ void widen(const Raw& r, float (&f)[8]) {
        f[0] = r.a.x; f[1] = r.a.y; f[2] = r.a.z; f[3] = r.a.w; f[4] = r.b.x; f[5] = r.b.y; f[6] = r.b.z; f[7] = r.b.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&f)[8]) {
        reinterpret_cast<float4*>(p)[0] = make_float4(f[0], f[1], f[2], f[3]);
        reinterpret_cast<float4*>(p)[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
};

// KW > 0: kernel width known at compile time (weights of a kernel row held in registers, the
// slide fully unrolled); KW == 0: any width up to kConvMaxKw, weights re-read per use.
template <typename T, int KW>
__global__ void __launch_bounds__(256)
dwconv3d_kernel(const T* __restrict__ x, const float* __restrict__ weight, const float* __restrict__ bias,
                T* __restrict__ y, int Tn, int H, int W, int C, int kt, int kh, int kw_rt) {
    const int kw = KW > 0 ? KW : kw_rt;
    const int cvecs = C / 8;
    const int xruns = (W + kConvRX - 1) / kConvRX;
    const long long total = static_cast<long long>(Tn) * H * xruns * cvecs;
    const long long id = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (id >= total) return;
    const int cv = static_cast<int>(id % cvecs);
    long long rest = id / cvecs;
    const int xr = static_cast<int>(rest % xruns); rest /= xruns;
    const int yy = static_cast<int>(rest % H);
    const int tt = static_cast<int>(rest / H);
    const int c0 = cv * 8, x0 = xr * kConvRX;

    float acc[kConvRX][8];
#pragma unroll
    for (int r = 0; r < kConvRX; ++r)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[r][e] = bias ? __ldg(bias + c0 + e) : 0.0f;

    for (int i = 0; i < kt; ++i) {
        const int st = tt + i - kt / 2;
        if (st < 0 || st >= Tn) continue;
        for (int j = 0; j < kh; ++j) {
            const int sy = yy + j - kh / 2;
            if (sy < 0 || sy >= H) continue;
            const T* row = x + (static_cast<long long>(st) * H + sy) * W * C + c0;
            const float* wrow = weight + static_cast<long long>((i * kh + j) * kw) * C + c0;
            if constexpr (KW > 0) {
                float wv[KW][8];
#pragma unroll
                for (int l = 0; l < KW; ++l) {
                    const float4 wa = __ldg(reinterpret_cast<const float4*>(wrow + static_cast<long long>(l) * C));
                    const float4 wb = __ldg(reinterpret_cast<const float4*>(wrow + static_cast<long long>(l) * C) + 1);
                    wv[l][0] = wa.x; wv[l][1] = wa.y; wv[l][2] = wa.z; wv[l][3] = wa.w;
                    wv[l][4] = wb.x; wv[l][5] = wb.y; wv[l][6] = wb.z; wv[l][7] = wb.w;
                }
                // all input vectors of this kernel row first (RX + KW - 1 independent loads in
                // flight), then the slide
                typename Vec8<T>::Raw raw[KW + kConvRX - 1];
#pragma unroll
                for (int s = 0; s < KW + kConvRX - 1; ++s) {
                    const int sx = x0 + s - KW / 2;
                    raw[s] = (sx >= 0 && sx < W) ? Vec8<T>::load_raw(row + static_cast<long long>(sx) * C)
                                                 : Vec8<T>::zero_raw();
                }
#pragma unroll
                for (int s = 0; s < KW + kConvRX - 1; ++s) {
                    float in[8];
                    Vec8<T>::widen(raw[s], in);
#pragma unroll
                    for (int r = 0; r < kConvRX; ++r) {
                        const int l = s - r;                      // tap that maps input s to output r
                        if (l < 0 || l >= KW) continue;
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[r][e] = fmaf(wv[l][e], in[e], acc[r][e]);
                    }
                }
            } else {
                for (int s = 0; s < kw + kConvRX - 1; ++s) {
                    const int sx = x0 + s - kw / 2;
                    if (sx < 0 || sx >= W) continue;
                    float in[8];
                    Vec8<T>::load(row + static_cast<long long>(sx) * C, in);
#pragma unroll
                    for (int r = 0; r < kConvRX; ++r) {
                        const int l = s - r;
                        if (l < 0 || l >= kw) continue;
                        const float4 wa = __ldg(reinterpret_cast<const float4*>(wrow + static_cast<long long>(l) * C));
                        const float4 wb = __ldg(reinterpret_cast<const float4*>(wrow + static_cast<long long>(l) * C) + 1);
                        const float wv[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[r][e] = fmaf(wv[e], in[e], acc[r][e]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kConvRX; ++r) {
        const int ox = x0 + r;
        if (ox < W) Vec8<T>::store(y + ((static_cast<long long>(tt) * H + yy) * W + ox) * C + c0, acc[r]);
    }
}

template <typename T>
void launch_dwconv(const void* x, const float* weight, const float* bias, void* y, int T_, int H, int W, int C,
                   const int kernel[3], unsigned blocks, cudaStream_t st) {
    const T* xp = static_cast<const T*>(x);
    T* yp = static_cast<T*>(y);
#define DSA3D_CONV_CASE(KW) \
    case KW: dwconv3d_kernel<T, KW><<<blocks, 256, 0, st>>>(xp, weight, bias, yp, T_, H, W, C, kernel[0], kernel[1], KW); break;
    switch (kernel[2]) {
        DSA3D_CONV_CASE(1)
        DSA3D_CONV_CASE(3)
        DSA3D_CONV_CASE(5)
        DSA3D_CONV_CASE(7)
        default: dwconv3d_kernel<T, 0><<<blocks, 256, 0, st>>>(xp, weight, bias, yp, T_, H, W, C, kernel[0], kernel[1], kernel[2]);
    }
#undef DSA3D_CONV_CASE
}

// ------------------------------------------------------------------------------------------
// Linear layer on tensor cores.
// ------------------------------------------------------------------------------------------
constexpr int BM = 128, BK = 64, kStages = 4, kMaxBN = 256;
constexpr int kGemmThreads = 192;                 // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue

struct __align__(1024) GemmSmem {
    __nv_bfloat16 a[kStages][BM * BK];
    __nv_bfloat16 b[kStages][kMaxBN * BK];
    uint64_t full[kStages], empty[kStages], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
offsets_gemm_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_w,
                    const float* __restrict__ bias, float* __restrict__ out, long long M, int N, int K, int BN,
                    long long m_tiles, int n_tiles) {
    extern __shared__ unsigned char raw[];
    GemmSmem& s = *reinterpret_cast<GemmSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kblocks = (K + BK - 1) / BK;
    const long long tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(smem_u32(&s.full[i]), 1); mbar_init(smem_u32(&s.empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&s.acc_full[i]), 1); mbar_init(smem_u32(&s.acc_empty[i]), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {                               // both accumulator buffers: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(2 * kMaxBN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;                       // k-block counter across tiles: stage and phase
            for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
                const int n0 = static_cast<int>(tile % n_tiles) * BN;
                const long long m0 = (tile / n_tiles) * BM;
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int st = it % kStages;
                    if (!mbar_wait(smem_u32(&s.empty[st]), ((it / kStages) & 1) ^ 1)) { ok = false; break; }
                    mbar_expect_tx(smem_u32(&s.full[st]), static_cast<uint32_t>((BM + BN) * BK * 2));
                    tma_load_2d(smem_u32(s.a[st]), &map_u, smem_u32(&s.full[st]), kb * BK, static_cast<int>(m0));
                    tma_load_2d(smem_u32(s.b[st]), &map_w, smem_u32(&s.full[st]), kb * BK, n0);
                }
                if (!ok) { atomicExch(&g_timeout_flag, 1); break; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                   (static_cast<uint32_t>(BM >> 4) << 24);   // fp32 accumulate, bf16 x bf16, K-major
            uint32_t it = 0, local = 0;
            bool ok = true;
            for (long long tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++local) {
                const uint32_t buf = local & 1;
                if (!mbar_wait(smem_u32(&s.acc_empty[buf]), ((local >> 1) & 1) ^ 1)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem + buf * kMaxBN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int st = it % kStages;
                    if (!mbar_wait(smem_u32(&s.full[st]), (it / kStages) & 1)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t da = smem_desc(smem_u32(s.a[st])), db = smem_desc(smem_u32(s.b[st]));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)                         // 16 channels = 32 bytes per step
                        umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
                    umma_commit(smem_u32(&s.empty[st]));                      // stage free once these MMAs have read it
                }
                umma_commit(smem_u32(&s.acc_full[buf]));
            }
            if (!ok) atomicExch(&g_timeout_flag, 2);
        }
    } else {
        const int quarter = warp & 3;                 // the 32 TMEM lanes this warp can read
        uint32_t local = 0;
        for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++local) {
            const uint32_t buf = local & 1;
            const int n0 = static_cast<int>(tile % n_tiles) * BN;
            const long long row = (tile / n_tiles) * BM + quarter * 32 + lane;
            if (!mbar_wait(smem_u32(&s.acc_full[buf]), (local >> 1) & 1)) {
                if (lane == 0) atomicExch(&g_timeout_flag, 3);
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_load_32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN + c0, r);
                if (row < M) {
                    float* dst = out + row * N + n0 + c0;
                    if (n0 + c0 + 32 <= N && (N & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 b4 = __ldg(reinterpret_cast<const float4*>(bias + n0 + c0 + j));
                            *reinterpret_cast<float4*>(dst + j) =
                                make_float4(__uint_as_float(r[j]) + b4.x, __uint_as_float(r[j + 1]) + b4.y,
                                            __uint_as_float(r[j + 2]) + b4.z, __uint_as_float(r[j + 3]) + b4.w);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c0 + j < N) dst[j] = __uint_as_float(r[j]) + __ldg(bias + n0 + c0 + j);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.acc_empty[buf]));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kMaxBN));
}

// ------------------------------------------------------------------------------------------
// Depthwise convolution, bf16, staged through shared memory by TMA.  A CTA owns a column of
// the grid - TY x TX positions, 64 channels (one 128-byte row per position) - and marches
// along t.  Each input plane of the column (with its kh-1 / kw-1 halo, zero-filled by the
// TMA unit outside the grid) is fetched once into a ring of kt+1 shared-memory slots, one
// plane ahead of the arithmetic; a thread produces 4 outputs along x for 8 channels and
// slides the kernel row over kw+3 shared-memory vectors held in registers.
// ------------------------------------------------------------------------------------------
constexpr int kCvTY = 4, kCvTX = 16, kCvRX = 4, kCvCh = 64, kCvThreads = 128, kCvMaxKt = 7;

template <int KW>
__global__ void __launch_bounds__(kCvThreads)
dwconv3d_tma_kernel(const __grid_constant__ CUtensorMap map_x, const float* __restrict__ weight,
                    const float* __restrict__ bias, __nv_bfloat16* __restrict__ y, int Tn, int H, int W, int C,
                    int kt, int kh, int t_chunk) {
    extern __shared__ unsigned char raw_smem[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(raw_smem) + 127) & ~uintptr_t(127));
    const int ring = kt + 1;
    const int ph = kCvTY + kh - 1, pw = kCvTX + KW - 1;                 // plane extent with halo
    const uint32_t plane_bytes = static_cast<uint32_t>(ph * pw * kCvCh * 2);
    float* wsm = reinterpret_cast<float*>(base + static_cast<size_t>(ring) * plane_bytes);   // [taps][64]
    uint64_t* bars = reinterpret_cast<uint64_t*>(wsm + kt * kh * KW * kCvCh);                 // [ring]

    const int tid = threadIdx.x;
    const int cv = tid & 7, xg = (tid >> 3) & 3, yl = tid >> 5;         // 8 channel vectors x 4 x-groups x 4 rows
    const int c0 = blockIdx.x * kCvCh;
    const int tiles_x = (W + kCvTX - 1) / kCvTX;
    const int x0 = (blockIdx.y % tiles_x) * kCvTX, y0 = (blockIdx.y / tiles_x) * kCvTY;
    const int t_begin = blockIdx.z * t_chunk, t_end = min(Tn, t_begin + t_chunk);
    const int lo = kt / 2;                                              // planes t-lo .. t-lo+kt-1 feed output t

    // per tap: the first four channels of every 8-channel vector, then the last four, so that
    // the 8 lanes of a quarter-warp read 128 contiguous bytes (no bank conflicts)
    for (int i = tid; i < kt * kh * KW * kCvCh; i += kCvThreads) {
        const int tap = i / kCvCh, ch = i % kCvCh;
        wsm[tap * kCvCh + ((ch >> 2) & 1) * 32 + (ch >> 3) * 4 + (ch & 3)] =
            __ldg(weight + static_cast<long long>(tap) * C + c0 + ch);
    }
    if (tid == 0) {
        for (int i = 0; i < ring; ++i) mbar_init(smem_u32(&bars[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // plane index n = p - (t_begin - lo) counts the planes of this CTA from 0; slot n % ring
    auto issue = [&](int n) {
        const int p = t_begin - lo + n, slot = n % ring;
        mbar_expect_tx(smem_u32(&bars[slot]), plane_bytes);
        tma_load_4d(smem_u32(base + static_cast<size_t>(slot) * plane_bytes), &map_x, smem_u32(&bars[slot]), c0,
                    x0 - KW / 2, y0 - kh / 2, p);
    };
    if (tid == 0)
        for (int n = 0; n < kt; ++n) issue(n);

    float bias_v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) bias_v[e] = bias ? __ldg(bias + c0 + cv * 8 + e) : 0.0f;
    const int oy = y0 + yl, ox0 = x0 + xg * kCvRX;
    bool ok = true;

    for (int t = t_begin; t < t_end && ok; ++t) {
        const int n_last = t - t_begin + kt - 1;                        // newest plane output t needs
        if (tid == 0 && t + 1 < t_end) issue(n_last + 1);              // its slot was last read by output t-1
        // the first output waits for all of its kt planes, later ones only for the newest
        for (int n = (t == t_begin ? n_last - (kt - 1) : n_last); n <= n_last; ++n)
            if (!mbar_wait(smem_u32(&bars[n % ring]), (n / ring) & 1)) {
                atomicExch(&g_timeout_flag, 4);
                ok = false;
                break;
            }
        float acc[kCvRX][8];
#pragma unroll
        for (int r = 0; r < kCvRX; ++r)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[r][e] = bias_v[e];
        if (ok) {
            for (int i = 0; i < kt; ++i) {
                const int n = t - t_begin + i;                          // plane t - lo + i
                const unsigned char* plane = base + static_cast<size_t>(n % ring) * plane_bytes;
                for (int j = 0; j < kh; ++j) {
                    const unsigned char* row = plane + (static_cast<size_t>(yl + j) * pw + xg * kCvRX) * (kCvCh * 2) + cv * 16;
                    const float* wrow = wsm + (i * kh + j) * KW * kCvCh + cv * 4;
                    float wv[KW][8];
#pragma unroll
                    for (int l = 0; l < KW; ++l) {
                        const float4 wa = *reinterpret_cast<const float4*>(wrow + l * kCvCh);
                        const float4 wb = *reinterpret_cast<const float4*>(wrow + l * kCvCh + 32);
                        wv[l][0] = wa.x; wv[l][1] = wa.y; wv[l][2] = wa.z; wv[l][3] = wa.w;
                        wv[l][4] = wb.x; wv[l][5] = wb.y; wv[l][6] = wb.z; wv[l][7] = wb.w;
                    }
                    uint4 in_raw[KW + kCvRX - 1];
#pragma unroll
                    for (int s = 0; s < KW + kCvRX - 1; ++s)
                        in_raw[s] = *reinterpret_cast<const uint4*>(row + s * (kCvCh * 2));
#pragma unroll
                    for (int s = 0; s < KW + kCvRX - 1; ++s) {
                        float in[8];
                        Vec8<__nv_bfloat16>::widen(in_raw[s], in);
#pragma unroll
                        for (int r = 0; r < kCvRX; ++r) {
                            const int l = s - r;
                            if (l < 0 || l >= KW) continue;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[r][e] = fmaf(wv[l][e], in[e], acc[r][e]);
                        }
                    }
                }
            }
            if (oy < H) {
#pragma unroll
                for (int r = 0; r < kCvRX; ++r)
                    if (ox0 + r < W)
                        Vec8<__nv_bfloat16>::store(
                            y + ((static_cast<long long>(t) * H + oy) * W + ox0 + r) * C + c0 + cv * 8, acc[r]);
            }
        }
        __syncthreads();                                                // plane t - lo may now be overwritten
    }
}

// The same contraction by pairs of CTAs (a cluster of two SMs on one 256 x BN tile,
// tcgen05.mma.cta_group::2): each CTA loads its own 128 rows of u and HALF of the w tile, the
// leader's single MMA thread multiplies both CTAs' operands and its commits arrive on the
// barriers of both, each CTA drains its own 128 accumulator rows.  Halving the w traffic per SM
// takes the operand stream under the 64 B/clk an SM can pull from L2 (the one-CTA tiling needs
// 93 B/clk at full tensor rate).
constexpr int kPairStages = 6;
struct __align__(1024) GemmPairSmem {
    __nv_bfloat16 a[kPairStages][BM * BK];
    __nv_bfloat16 b[kPairStages][(kMaxBN / 2) * BK];
    uint64_t full[kPairStages], empty[kPairStages], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
offsets_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_w,
                         const float* __restrict__ bias, float* __restrict__ out, long long M, int N, int K, int BN,
                         long long m_tiles, int n_tiles) {
    extern __shared__ unsigned char raw[];
    GemmPairSmem& s = *reinterpret_cast<GemmPairSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                       // 0: leader (issues the MMAs)
    const int kblocks = (K + BK - 1) / BK;
    const long long tiles = m_tiles * n_tiles;                  // m_tiles counts 256-row tiles here
    const long long pair = blockIdx.x / 2, pairs = gridDim.x / 2;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kPairStages; ++i) { mbar_init(smem_u32(&s.full[i]), 1); mbar_init(smem_u32(&s.empty[i]), 1); }
        // acc_empty of the leader collects the four epilogue warps of both CTAs
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&s.acc_full[i]), 1); mbar_init(smem_u32(&s.acc_empty[i]), 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(2 * kMaxBN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                          // both CTAs' barriers exist from here on
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            for (long long tile = pair; tile < tiles; tile += pairs) {
                const int n0 = static_cast<int>(tile % n_tiles) * BN;
                const long long m0 = (tile / n_tiles) * (2 * BM);
                bool ok = true;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int st = it % kPairStages;
                    if (!mbar_wait(smem_u32(&s.empty[st]), ((it / kPairStages) & 1) ^ 1)) { ok = false; break; }
                    const uint32_t full_leader = map_to_cta(smem_u32(&s.full[st]), 0);
                    if (rank == 0)                               // the bytes of both CTAs land on the leader's barrier
                        mbar_expect_tx(smem_u32(&s.full[st]), static_cast<uint32_t>(2 * (BM + BN / 2) * BK * 2));
                    tma_load_2d_pair(smem_u32(s.a[st]), &map_u, full_leader, kb * BK,
                                     static_cast<int>(m0) + static_cast<int>(rank) * BM);
                    tma_load_2d_pair(smem_u32(s.b[st]), &map_w, full_leader, kb * BK, n0 + static_cast<int>(rank) * (BN / 2));
                }
                if (!ok) { atomicExch(&g_timeout_flag, 8); break; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                   (static_cast<uint32_t>((2 * BM) >> 4) << 24);
            uint32_t it = 0, local = 0;
            bool ok = true;
            for (long long tile = pair; tile < tiles && ok; tile += pairs, ++local) {
                const uint32_t buf = local & 1;
                if (!mbar_wait(smem_u32(&s.acc_empty[buf]), ((local >> 1) & 1) ^ 1)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem + buf * kMaxBN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int st = it % kPairStages;
                    if (!mbar_wait(smem_u32(&s.full[st]), (it / kPairStages) & 1)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t da = smem_desc(smem_u32(s.a[st])), db = smem_desc(smem_u32(s.b[st]));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
                    umma_commit_pair(smem_u32(&s.empty[st]));          // frees the stage in both CTAs
                }
                umma_commit_pair(smem_u32(&s.acc_full[buf]));
            }
            if (!ok) atomicExch(&g_timeout_flag, 9);
        }
    } else {
        const int quarter = warp & 3;
        uint32_t local = 0;
        for (long long tile = pair; tile < tiles; tile += pairs, ++local) {
            const uint32_t buf = local & 1;
            const int n0 = static_cast<int>(tile % n_tiles) * BN;
            const long long row = (tile / n_tiles) * (2 * BM) + rank * BM + quarter * 32 + lane;
            if (!mbar_wait(smem_u32(&s.acc_full[buf]), (local >> 1) & 1)) {
                if (lane == 0) atomicExch(&g_timeout_flag, 10);
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_load_32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN + c0, r);
                if (row < M) {
                    float* dst = out + row * N + n0 + c0;
                    if (n0 + c0 + 32 <= N && (N & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 b4 = __ldg(reinterpret_cast<const float4*>(bias + n0 + c0 + j));
                            *reinterpret_cast<float4*>(dst + j) =
                                make_float4(__uint_as_float(r[j]) + b4.x, __uint_as_float(r[j + 1]) + b4.y,
                                            __uint_as_float(r[j + 2]) + b4.z, __uint_as_float(r[j + 3]) + b4.w);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c0 + j < N) dst[j] = __uint_as_float(r[j]) + __ldg(bias + n0 + c0 + j);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&s.acc_empty[buf]), 0));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                          // neither CTA leaves while its peer may still signal it
    if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kMaxBN));
}

// fp32 storage: one thread per output, plain fp32 FMAs in channel order.
__global__ void __launch_bounds__(256)
offsets_linear_f32_kernel(const float* __restrict__ u, const float* __restrict__ w, const float* __restrict__ bias,
                          float* __restrict__ out, long long M, int N, int K) {
    const long long id = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (id >= M * N) return;
    const long long m = id / N;
    const int n = static_cast<int>(id - m * N);
    const float* ur = u + m * K;
    const float* wr = w + static_cast<long long>(n) * K;
    float acc = 0.0f;
    for (int c = 0; c < K; ++c) acc = fmaf(__ldg(ur + c), __ldg(wr + c), acc);
    out[id] = acc + (bias ? __ldg(bias + n) : 0.0f);
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &res) == cudaSuccess &&
            res == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Row-major [rows, cols] bf16 matrix, tiles of box_rows x 64 columns, 128-byte swizzle, zero fill
// outside the matrix.
bool make_map(CUtensorMap* map, const void* ptr, unsigned long long rows, unsigned long long cols, unsigned box_rows) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Channels-last activations [T, H, W, C] bf16 as a 4-D map with boxes of 64 channels x pw x ph x 1.
bool make_map_activations(CUtensorMap* map, const void* ptr, int T, int H, int W, int C, int pw, int ph) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(H),
                                static_cast<cuuint64_t>(T)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(C) * 2, static_cast<cuuint64_t>(W) * C * 2,
                                   static_cast<cuuint64_t>(H) * W * C * 2};
    const cuuint32_t box[4] = {kCvCh, static_cast<cuuint32_t>(pw), static_cast<cuuint32_t>(ph), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch the staged kernel if the shape suits it; returns false when the caller should use the
// plain kernel instead (fp32, odd channel counts, wide kernels).  *err receives a launch error.
bool try_dwconv_tma(const void* x, const float* weight, const float* bias, void* y, int T, int H, int W, int C,
                    const int kernel[3], cudaStream_t st, cudaError_t* err) {
    *err = cudaSuccess;
    const int kt = kernel[0], kh = kernel[1], kw = kernel[2];
    if (C % kCvCh || kt > kCvMaxKt || (kw != 1 && kw != 3 && kw != 5 && kw != 7)) return false;
    const int ph = kCvTY + kh - 1, pw = kCvTX + kw - 1;
    if (ph > 256 || pw > 256) return false;
    const size_t plane = static_cast<size_t>(ph) * pw * kCvCh * 2;
    const size_t smem = 128 + (kt + 1) * plane + static_cast<size_t>(kt) * kh * kw * kCvCh * 4 + (kt + 1) * 8;
    if (smem > 200 * 1024) return false;
    CUtensorMap map;
    if (!make_map_activations(&map, x, T, H, W, C, pw, ph)) return false;
    const int tiles = ((W + kCvTX - 1) / kCvTX) * ((H + kCvTY - 1) / kCvTY);
    if (tiles > 65535) return false;
    // split t so that the grid fills the GPU a few times over, but keep chunks long enough to
    // amortise the kt-1 planes of run-in
    int splits = 1;
    const long long columns = static_cast<long long>(C / kCvCh) * tiles;
    while (columns * splits < 148 * 8 && T / (splits * 2) >= 4 * kt) splits *= 2;
    const int t_chunk = (T + splits - 1) / splits;
    const dim3 grid(C / kCvCh, tiles, (T + t_chunk - 1) / t_chunk);
#define DSA3D_CONV_TMA_CASE(KW)                                                                                    \
    case KW:                                                                                                       \
        *err = cudaFuncSetAttribute(dwconv3d_tma_kernel<KW>, cudaFuncAttributeMaxDynamicSharedMemorySize,          \
                                    static_cast<int>(smem));                                                       \
        if (*err == cudaSuccess) {                                                                                 \
            dwconv3d_tma_kernel<KW><<<grid, kCvThreads, smem, st>>>(map, weight, bias, static_cast<__nv_bfloat16*>(y), \
                                                                    T, H, W, C, kt, kh, t_chunk);                  \
            *err = cudaGetLastError();                                                                             \
        }                                                                                                          \
        break;
    switch (kw) {
        DSA3D_CONV_TMA_CASE(1)
        DSA3D_CONV_TMA_CASE(3)
        DSA3D_CONV_TMA_CASE(5)
        DSA3D_CONV_TMA_CASE(7)
    }
#undef DSA3D_CONV_TMA_CASE
    return true;
}

}  // namespace

bool dsa3d::encode_tensor_map_bf16(CUtensorMap* map, const void* base, int rank, const unsigned long long* dims,
                                   const unsigned long long* strides_bytes, const unsigned* box, bool swizzle128) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc || rank < 1 || rank > 5) return false;
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base), d, st, b,
               es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int* dsa3d::timeout_flag_device_address() {
    void* p = nullptr;
    return cudaGetSymbolAddress(&p, g_timeout_flag) == cudaSuccess ? static_cast<int*>(p) : nullptr;
}

namespace {

int cuda_failed(cudaError_t e) { return dsa3d::note_cuda_error(e); }

}  // namespace

extern "C" {

int dsa3d_dwconv3d_forward(const void* x, const float* weight, const float* bias, int T, int H, int W, int C,
                           const int kernel[3], void* y, int dtype, void* stream) {
    if (!x || !weight || !y || !kernel) return DSA3D_ERR_NULL_POINTER;
    if (T < 1 || H < 1 || W < 1 || C < 8 || C % 8) return DSA3D_ERR_BAD_SHAPE;
    if (kernel[0] < 1 || kernel[1] < 1 || kernel[2] < 1 || kernel[2] > kConvMaxKw || kernel[0] > 15 || kernel[1] > 15)
        return DSA3D_ERR_BAD_SHAPE;
    if (dtype != DSA3D_F32 && dtype != DSA3D_BF16) return DSA3D_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(y) || !aligned16(weight) || (bias && !aligned16(bias))) return DSA3D_ERR_MISALIGNED;
    const long long total = static_cast<long long>(T) * H * ((W + kConvRX - 1) / kConvRX) * (C / 8);
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return DSA3D_ERR_BAD_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == DSA3D_BF16) {
        cudaError_t te;
        if (try_dwconv_tma(x, weight, bias, y, T, H, W, C, kernel, st, &te))
            return te == cudaSuccess ? DSA3D_OK : cuda_failed(te);
    }
    if (dtype == DSA3D_BF16)
        launch_dwconv<__nv_bfloat16>(x, weight, bias, y, T, H, W, C, kernel, static_cast<unsigned>(blocks), st);
    else
        launch_dwconv<float>(x, weight, bias, y, T, H, W, C, kernel, static_cast<unsigned>(blocks), st);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

int dsa3d_offsets_linear_forward(const void* u, const void* w, const float* bias, long long tokens, int C, int O,
                                 float* offsets, int dtype, void* stream) {
    if (!u || !w || !bias || !offsets) return DSA3D_ERR_NULL_POINTER;
    if (tokens < 1 || C < 8 || C % 8 || O < 1 || tokens > 0x7fffffffLL) return DSA3D_ERR_BAD_SHAPE;
    if (dtype != DSA3D_F32 && dtype != DSA3D_BF16) return DSA3D_ERR_UNSUPPORTED;
    if (!aligned16(u) || !aligned16(w) || !aligned16(bias) || !aligned16(offsets)) return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == DSA3D_F32) {
        const long long blocks = (tokens * O + 255) / 256;
        if (blocks > 0x7fffffffLL) return DSA3D_ERR_BAD_SHAPE;
        offsets_linear_f32_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(
            static_cast<const float*>(u), static_cast<const float*>(w), bias, offsets, tokens, O, C);
        const cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
    }
    // column tiles of equal width, a multiple of 32 columns, at most 256
    const int n_tiles = (O + kMaxBN - 1) / kMaxBN;
    const int BN = ((O + n_tiles - 1) / n_tiles + 31) / 32 * 32;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_failed(e);
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_failed(e);
    CUtensorMap map_u, map_w;
    const bool pair = sms >= 2 && !std::getenv("DSA3D_GEMM_ONE_CTA");     // pairs of CTAs unless switched off
    if (pair) {
        const long long m_tiles = (tokens + 2 * BM - 1) / (2 * BM);
        if (!make_map(&map_u, u, static_cast<unsigned long long>(tokens), static_cast<unsigned long long>(C), BM) ||
            !make_map(&map_w, w, static_cast<unsigned long long>(O), static_cast<unsigned long long>(C),
                      static_cast<unsigned>(BN / 2)))
            return DSA3D_ERR_UNSUPPORTED;
        const size_t smem = sizeof(GemmPairSmem) + 1024;
        e = cudaFuncSetAttribute(offsets_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem));
        if (e != cudaSuccess) return cuda_failed(e);
        const long long tiles = m_tiles * n_tiles;
        const long long want = 2 * (tiles < sms / 2 ? tiles : sms / 2);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(want));
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, offsets_gemm_pair_kernel, map_u, map_w, bias, offsets, tokens, O, C, BN, m_tiles,
                               n_tiles);
        return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
    }
    const long long m_tiles = (tokens + BM - 1) / BM;
    if (!make_map(&map_u, u, static_cast<unsigned long long>(tokens), static_cast<unsigned long long>(C), BM) ||
        !make_map(&map_w, w, static_cast<unsigned long long>(O), static_cast<unsigned long long>(C),
                  static_cast<unsigned>(BN)))
        return DSA3D_ERR_UNSUPPORTED;
    const size_t smem = sizeof(GemmSmem) + 1024;
    e = cudaFuncSetAttribute(offsets_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_failed(e);
    const long long tiles = m_tiles * n_tiles;
    const int grid = static_cast<int>(tiles < sms ? tiles : sms);
    offsets_gemm_kernel<<<grid, kGemmThreads, smem, st>>>(map_u, map_w, bias, offsets, tokens, O, C, BN, m_tiles,
                                                           n_tiles);
    e = cudaGetLastError();
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

int dsa3d_device_timeout_flag(void) {
    int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_timeout_flag, sizeof(int)) != cudaSuccess) return -1;
    return flag;
}

}  // extern "C"
