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
#include <type_traits>

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
                T* __restrict__ y, int Tn, int H, int W, int C, int kt, int kh, int kw_rt, int ct, int chh, int cw) {
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
        const int st = tt + i - ct;
        if (st < 0 || st >= Tn) continue;
        for (int j = 0; j < kh; ++j) {
            const int sy = yy + j - chh;
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
                    const int sx = x0 + s - cw;
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
                    const int sx = x0 + s - cw;
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
                   const int kernel[3], const int centre[3], unsigned blocks, cudaStream_t st) {
    const T* xp = static_cast<const T*>(x);
    T* yp = static_cast<T*>(y);
#define DSA3D_CONV_CASE(KW) \
    case KW: dwconv3d_kernel<T, KW><<<blocks, 256, 0, st>>>(xp, weight, bias, yp, T_, H, W, C, kernel[0], kernel[1], KW, \
                                                            centre[0], centre[1], centre[2]); break;
    switch (kernel[2]) {
        DSA3D_CONV_CASE(1)
        DSA3D_CONV_CASE(3)
        DSA3D_CONV_CASE(5)
        DSA3D_CONV_CASE(7)
        default: dwconv3d_kernel<T, 0><<<blocks, 256, 0, st>>>(xp, weight, bias, yp, T_, H, W, C, kernel[0], kernel[1], kernel[2],
                                                               centre[0], centre[1], centre[2]);
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
                    int kt, int kh, int t_chunk, int ct, int chh, int cw) {
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
    const int lo = ct;                                                  // planes t-lo .. t-lo+kt-1 feed output t

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
                    x0 - cw, y0 - chh, p);
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
        ok = __syncthreads_and(ok);                                     // all threads stop together or not at all
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
// what the epilogue does with the fp32 accumulators: out = acc + bias in fp32 (bias required);
// out = acc in bf16; out += acc
constexpr int kGemmStoreF32 = 0, kGemmStoreBf16 = 1, kGemmAddF32 = 2;
struct __align__(1024) GemmPairSmem {
    __nv_bfloat16 a[kPairStages][BM * BK];
    __nv_bfloat16 b[kPairStages][(kMaxBN / 2) * BK];
    float stage_out[4][2][32 * 32];        // per epilogue warp: two 32 x 32 fp32 boxes for TMA stores
    uint64_t full[kPairStages], empty[kPairStages], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

// MN_MAJOR: the operands are given as [K, M] and [K, N] row-major matrices (the contraction index
// is the row), fetched as boxes of 64 columns x BK rows; BN is 256 then.
template <int MODE, bool MN_MAJOR>
__global__ void __launch_bounds__(kGemmThreads, 1)
offsets_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_w,
                         const __grid_constant__ CUtensorMap map_out, int tma_store,
                         const float* __restrict__ bias, void* __restrict__ out_raw, long long M, int N, int K, int BN,
                         long long m_tiles, int n_tiles, int ksplits) {
    extern __shared__ unsigned char raw[];
    GemmPairSmem& s = *reinterpret_cast<GemmPairSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                       // 0: leader (issues the MMAs)
    const int kblocks = (K + BK - 1) / BK;
    // a work unit is one 256 x BN output tile (m_tiles counts 256-row tiles) times one of
    // `ksplits` equal ranges of k-blocks; the k-range is the slow index, so the units in flight at any
    // time are different tiles walking through the same k-range: each operand block is fetched from
    // DRAM once and found in L2 by the other tiles of its row or column
    const long long tiles = m_tiles * n_tiles * ksplits;
    auto k_range = [&](long long unit, int& kb0, int& kb1) {
        const int ks = static_cast<int>(unit / (m_tiles * n_tiles));
        kb0 = static_cast<int>(static_cast<long long>(kblocks) * ks / ksplits);
        kb1 = static_cast<int>(static_cast<long long>(kblocks) * (ks + 1) / ksplits);
    };
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
            for (long long unit = pair; unit < tiles; unit += pairs) {
                const long long tile = unit % (m_tiles * n_tiles);
                const int n0 = static_cast<int>(tile % n_tiles) * BN;
                const long long m0 = (tile / n_tiles) * (2 * BM);
                int kb0, kb1;
                k_range(unit, kb0, kb1);
                bool ok = true;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int st = it % kPairStages;
                    if (!mbar_wait(smem_u32(&s.empty[st]), ((it / kPairStages) & 1) ^ 1)) { ok = false; break; }
                    const uint32_t full_leader = map_to_cta(smem_u32(&s.full[st]), 0);
                    if (rank == 0)                               // the bytes of both CTAs land on the leader's barrier
                        mbar_expect_tx(smem_u32(&s.full[st]), static_cast<uint32_t>(2 * (BM + BN / 2) * BK * 2));
                    if constexpr (MN_MAJOR) {
                        const int ma = static_cast<int>(m0) + static_cast<int>(rank) * BM;
                        const int nb = n0 + static_cast<int>(rank) * (kMaxBN / 2);
#pragma unroll
                        for (int atom = 0; atom < 2; ++atom) {
                            tma_load_2d_pair(smem_u32(s.a[st]) + atom * (64 * BK * 2), &map_u, full_leader, ma + atom * 64,
                                             kb * BK);
                            tma_load_2d_pair(smem_u32(s.b[st]) + atom * (64 * BK * 2), &map_w, full_leader, nb + atom * 64,
                                             kb * BK);
                        }
                    } else {
                        tma_load_2d_pair(smem_u32(s.a[st]), &map_u, full_leader, kb * BK,
                                         static_cast<int>(m0) + static_cast<int>(rank) * BM);
                        tma_load_2d_pair(smem_u32(s.b[st]), &map_w, full_leader, kb * BK,
                                         n0 + static_cast<int>(rank) * (BN / 2));
                    }
                }
                if (!ok) { atomicExch(&g_timeout_flag, 8); break; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                                   (static_cast<uint32_t>((2 * BM) >> 4) << 24) |
                                   (MN_MAJOR ? (1u << 15) | (1u << 16) : 0u);       // both operands MN-major
            uint32_t it = 0, local = 0;
            bool ok = true;
            for (long long unit = pair; unit < tiles && ok; unit += pairs, ++local) {
                const uint32_t buf = local & 1;
                int kb0, kb1;
                k_range(unit, kb0, kb1);
                if (!mbar_wait(smem_u32(&s.acc_empty[buf]), ((local >> 1) & 1) ^ 1)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem + buf * kMaxBN;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int st = it % kPairStages;
                    if (!mbar_wait(smem_u32(&s.full[st]), (it / kPairStages) & 1)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if constexpr (MN_MAJOR) {
                        // 16 rows of 128 bytes per step: 2048 bytes = 128 in the descriptor's 16-byte units
                        const uint64_t da = smem_desc_mn(smem_u32(s.a[st]), 64 * BK * 2),
                                       db = smem_desc_mn(smem_u32(s.b[st]), 64 * BK * 2);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            umma_bf16_pair(d_tmem, da + 128 * k, db + 128 * k, idesc, ((kb - kb0) | k) ? 1u : 0u);
                    } else {
                        const uint64_t da = smem_desc(smem_u32(s.a[st])), db = smem_desc(smem_u32(s.b[st]));
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            umma_bf16_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, ((kb - kb0) | k) ? 1u : 0u);
                    }
                    umma_commit_pair(smem_u32(&s.empty[st]));          // frees the stage in both CTAs
                }
                umma_commit_pair(smem_u32(&s.acc_full[buf]));
            }
            if (!ok) atomicExch(&g_timeout_flag, 9);
        }
    } else {
        const int quarter = warp & 3;
        uint32_t local = 0, boxes = 0;
        for (long long unit = pair; unit < tiles; unit += pairs, ++local) {
            const uint32_t buf = local & 1;
            const long long tile = unit % (m_tiles * n_tiles);
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
                const bool whole = n0 + c0 + 32 <= N;
                if constexpr (MODE == kGemmStoreF32) {
                    if (tma_store) {
                        // the warp's 32 x 32 block goes through shared memory (128-byte rows, 16-byte
                        // chunks swizzled by the row as the tensor map expects) and out as one TMA box:
                        // whole 128-byte lines per row instead of 32 scattered 16-byte pieces per store
                        if (n0 + c0 >= N || row - lane >= M) continue;      // nothing of this box is inside
                        unsigned char* stg = reinterpret_cast<unsigned char*>(s.stage_out[quarter][boxes & 1]);
                        if (lane == 0) tma_store_wait_read<1>();           // the box before last has left this buffer
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float4 b4;
                            if (whole) {
                                b4 = __ldg(reinterpret_cast<const float4*>(bias + n0 + c0 + 4 * j));
                            } else {
                                const int cb = n0 + c0 + 4 * j;
                                b4 = make_float4(cb < N ? __ldg(bias + cb) : 0.f, cb + 1 < N ? __ldg(bias + cb + 1) : 0.f,
                                                 cb + 2 < N ? __ldg(bias + cb + 2) : 0.f, cb + 3 < N ? __ldg(bias + cb + 3) : 0.f);
                            }
                            *reinterpret_cast<float4*>(stg + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                make_float4(__uint_as_float(r[4 * j]) + b4.x, __uint_as_float(r[4 * j + 1]) + b4.y,
                                            __uint_as_float(r[4 * j + 2]) + b4.z, __uint_as_float(r[4 * j + 3]) + b4.w);
                        }
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0)
                            tma_store_2d(&map_out, smem_u32(stg), n0 + c0, static_cast<int>(row - lane));
                        ++boxes;
                        continue;
                    }
                    if (row >= M) continue;
                    float* dst = static_cast<float*>(out_raw) + row * N + n0 + c0;
                    if (whole && (N & 3) == 0) {
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
                } else if constexpr (MODE == kGemmStoreBf16) {
                    if (tma_store) {
                        // 32 rows x 64 bytes through shared memory (64-byte swizzle: the 16-byte chunk index
                        // is XORed with bits 1-2 of the row) and out as one TMA box
                        if (n0 + c0 >= N || row - lane >= M) continue;
                        unsigned char* stg = reinterpret_cast<unsigned char*>(s.stage_out[quarter][boxes & 1]);
                        if (lane == 0) tma_store_wait_read<1>();
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * j + 2 * e]),
                                                                               __uint_as_float(r[8 * j + 2 * e + 1]));
                                w[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(stg + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) =
                                make_uint4(w[0], w[1], w[2], w[3]);
                        }
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0)
                            tma_store_2d(&map_out, smem_u32(stg), n0 + c0, static_cast<int>(row - lane));
                        ++boxes;
                        continue;
                    }
                    if (row >= M) continue;
                    __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(out_raw) + row * N + n0 + c0;
                    if (whole && (N & 7) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[j + 2 * e]),
                                                                               __uint_as_float(r[j + 2 * e + 1]));
                                w[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c0 + j < N) dst[j] = __float2bfloat16_rn(__uint_as_float(r[j]));
                    }
                } else {                                     // kGemmAddF32: partial sums of a k-range
                    if (row >= M) continue;
                    float* dst = static_cast<float*>(out_raw) + row * N + n0 + c0;
                    if (whole && (N & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + j),
                                         "f"(__uint_as_float(r[j])), "f"(__uint_as_float(r[j + 1])),
                                         "f"(__uint_as_float(r[j + 2])), "f"(__uint_as_float(r[j + 3]))
                                         : "memory");
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c0 + j < N) atomicAdd(dst + j, __uint_as_float(r[j]));
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&s.acc_empty[buf]), 0));
        }
        if (MODE != kGemmAddF32 && tma_store && lane == 0) tma_store_wait_all();     // shared memory is read, stores done
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
bool make_map(CUtensorMap* map, const void* ptr, unsigned long long rows, unsigned long long cols, unsigned box_rows,
              unsigned long long ld = 0) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {(ld ? ld : cols) * 2};          // row pitch in bytes (a multiple of 16)
    const cuuint32_t box[2] = {BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major fp32 [rows, cols] output, boxes of 32 x 32, 128-byte swizzle (cols a multiple of 4).
bool make_map_out_f32(CUtensorMap* map, void* ptr, unsigned long long rows, unsigned long long cols) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major bf16 [rows, cols] output, boxes of 32 x 32 (64-byte rows), 64-byte swizzle (cols a multiple of 8).
bool make_map_out_bf16(CUtensorMap* map, void* ptr, unsigned long long rows, unsigned long long cols) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// out[M, N] = A[M, K] . B[N, K]^T on pairs of CTAs; A and B row-major bf16 with row pitches lda, ldb
// (elements, multiples of 8).  mode: what the epilogue does; ksplits: equal ranges of k-blocks per
// output tile (> 1 only with kGemmAddF32).  Column tiles of equal width, a multiple of 32, at most 256.
cudaError_t launch_pair_gemm(const void* A, unsigned long long lda, const void* B, unsigned long long ldb,
                             const float* bias, void* out, long long M, int N, int K, int mode, int ksplits, int sms,
                             cudaStream_t st, bool* unsupported, bool mn_major = false) {
    *unsupported = false;
    const int n_tiles = (N + kMaxBN - 1) / kMaxBN;
    const int BN = mn_major ? kMaxBN : ((N + n_tiles - 1) / n_tiles + 31) / 32 * 32;
    const long long m_tiles = (M + 2 * BM - 1) / (2 * BM);
    CUtensorMap map_a, map_b;
    // MN-major: A is [K, M] and B is [K, N] in memory, fetched as boxes of 64 columns x BK rows
    const bool ok = mn_major
        ? make_map(&map_a, A, static_cast<unsigned long long>(K), static_cast<unsigned long long>(M), BK, lda) &&
          make_map(&map_b, B, static_cast<unsigned long long>(K), static_cast<unsigned long long>(N), BK, ldb)
        : make_map(&map_a, A, static_cast<unsigned long long>(M), static_cast<unsigned long long>(K), BM, lda) &&
          make_map(&map_b, B, static_cast<unsigned long long>(N), static_cast<unsigned long long>(K),
                   static_cast<unsigned>(BN / 2), ldb);
    if (!ok || (mn_major && mode != kGemmAddF32)) {
        *unsupported = true;
        return cudaSuccess;
    }
    const size_t smem = sizeof(GemmPairSmem) + 1024;
    const long long units = m_tiles * n_tiles * ksplits;
    const long long want = 2 * (units < sms / 2 ? units : sms / 2);
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
    // fp32 + bias epilogue: 32 x 32 boxes by TMA when the rows of the output are 16-byte multiples
    CUtensorMap map_out = map_a;
    int tma_store = 0;
    if (mode == kGemmStoreF32 && (N & 3) == 0 && !std::getenv("DSA3D_GEMM_PLAIN_STORES") &&
        make_map_out_f32(&map_out, out, static_cast<unsigned long long>(M), static_cast<unsigned long long>(N)))
        tma_store = 1;
    if (mode == kGemmStoreBf16 && (N & 7) == 0 && !std::getenv("DSA3D_GEMM_PLAIN_STORES") &&
        make_map_out_bf16(&map_out, out, static_cast<unsigned long long>(M), static_cast<unsigned long long>(N)))
        tma_store = 1;
    auto launch = [&](auto kernel) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_out, tma_store, bias, out, M, N, K, BN, m_tiles, n_tiles,
                                  ksplits);
    };
    if (mn_major) return launch(offsets_gemm_pair_kernel<kGemmAddF32, true>);
    if (mode == kGemmStoreF32) return launch(offsets_gemm_pair_kernel<kGemmStoreF32, false>);
    if (mode == kGemmStoreBf16) return launch(offsets_gemm_pair_kernel<kGemmStoreBf16, false>);
    return launch(offsets_gemm_pair_kernel<kGemmAddF32, false>);
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

bool try_dwconv_333(const void* x, const float* weight, const float* bias, void* y, int T, int H, int W, int C,
                    const int centre[3], cudaStream_t st, cudaError_t* err);

// Launch the staged kernel if the shape suits it; returns false when the caller should use the
// plain kernel instead (fp32, odd channel counts, wide kernels).  *err receives a launch error.
bool try_dwconv_tma(const void* x, const float* weight, const float* bias, void* y, int T, int H, int W, int C,
                    const int kernel[3], const int centre[3], cudaStream_t st, cudaError_t* err) {
    *err = cudaSuccess;
    const int kt = kernel[0], kh = kernel[1], kw = kernel[2];
    if (C % kCvCh || kt > kCvMaxKt || (kw != 1 && kw != 3 && kw != 5 && kw != 7)) return false;
    if (kt == 3 && kh == 3 && kw == 3 && !std::getenv("DSA3D_CONV_GENERAL")) {
        cudaError_t e333;
        if (try_dwconv_333(x, weight, bias, y, T, H, W, C, centre, st, &e333)) {
            *err = e333;
            return true;
        }
    }
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
                                                                    T, H, W, C, kt, kh, t_chunk, centre[0],        \
                                                                    centre[1], centre[2]);                         \
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


// ------------------------------------------------------------------------------------------
// Backward of the two layers.
//   convolution:  dx = correlation of dy with the flipped kernel (the same kernels as the
//                 forward, centre kt-1-kt/2 etc.); dweight[tap, c] = sum_s x[s + disp] dy[s, c]
//                 and dbias by dwconv3d_wgrad_kernel.
//   linear layer: du = doffsets . w and dw = doffsets^T . u as two tensor-core contractions
//                 (bf16 operands: doffsets is rounded to bf16 once; the first takes a transposed
//                 copy of w so that both operands are K-major, the second reads doffsets and u
//                 as MN-major operands, the token index being their row), token slab by token
//                 slab; dbias from the fp32 doffsets.
// ------------------------------------------------------------------------------------------
__global__ void flip_weight_kernel(const float* __restrict__ w, float* __restrict__ wf, int taps, int C) {
    const long long id = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (id >= static_cast<long long>(taps) * C) return;
    const int tap = static_cast<int>(id / C), c = static_cast<int>(id % C);
    wf[static_cast<long long>(taps - 1 - tap) * C + c] = w[id];
}

template <typename T> struct Pair2;
template <> struct Pair2<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(const __nv_bfloat16* p) {
        const uint32_t r = __ldg(reinterpret_cast<const uint32_t*>(p));
        return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
    }
};
template <> struct Pair2<float> {
    static __device__ __forceinline__ float2 load(const float* p) { return __ldg(reinterpret_cast<const float2*>(p)); }
};

// One warp per (kernel row (i, j), chunk of grid rows); lane = a pair of neighbouring channels
// of a 64-channel group.  The warp marches along x over the input columns of its rows: one x
// vector per column feeds the kw taps of the kernel row against a sliding window of kw dy
// vectors held in registers.  The partial sums of a warp go to dweight with one atomic per
// (tap, channel); warps of a block are the kernel rows of the same grid rows, so they share
// their loads through L1.
constexpr int kWgradRows = 32;                  // grid rows (t, y) per warp
template <typename T, int KW>
__global__ void __launch_bounds__(1024)
dwconv3d_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dweight,
                      float* __restrict__ dbias, int Tn, int H, int W, int C, int kt, int kh, int kw_rt) {
    constexpr int MAXW = KW > 0 ? KW : kConvMaxKw;
    const int kw = KW > 0 ? KW : kw_rt;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const int c = blockIdx.x * 64 + lane * 2;
    if (c >= C) return;                                    // C is even: a pair is inside or outside
    const long long rows = static_cast<long long>(Tn) * H;
    const long long r0 = static_cast<long long>(blockIdx.y) * kWgradRows;
    const long long r1 = r0 + kWgradRows < rows ? r0 + kWgradRows : rows;
    const int ct = kt / 2, chh = kh / 2, cw = kw / 2;

    for (int ij = warp; ij < kt * kh; ij += warps) {
        const int i = ij / kh, j = ij % kh;
        float2 acc[MAXW];
#pragma unroll
        for (int l = 0; l < MAXW; ++l) acc[l] = make_float2(0.f, 0.f);
        float2 bsum = make_float2(0.f, 0.f);
        for (long long r = r0; r < r1; ++r) {
            const int tt = static_cast<int>(r / H), yy = static_cast<int>(r % H);
            const T* gy = dy + r * W * C + c;
            if (ij == 0 && dbias)
                for (int ox = 0; ox < W; ++ox) {
                    const float2 g = Pair2<T>::load(gy + static_cast<long long>(ox) * C);
                    bsum.x += g.x;
                    bsum.y += g.y;
                }
            const int st = tt + i - ct, sy = yy + j - chh;
            if (st < 0 || st >= Tn || sy < 0 || sy >= H) continue;
            const T* xr = x + (static_cast<long long>(st) * H + sy) * W * C + c;
            // window[l] = dy at output column sx + cw - l (zero outside the row)
            float2 win[MAXW];
#pragma unroll
            for (int l = 0; l < MAXW; ++l) win[l] = make_float2(0.f, 0.f);
            // before input column 0: outputs cw-l for l = 1 .. (shifted in below)
#pragma unroll
            for (int l = 1; l < MAXW; ++l) {
                const int ox = cw - l;                      // output column seen by tap l at sx = 0, minus the shift
                if (l < kw && ox >= 0 && ox < W) win[l] = Pair2<T>::load(gy + static_cast<long long>(ox) * C);
            }
#pragma unroll 4
            for (int sx = 0; sx < W; ++sx) {
                const int ox0 = sx + cw;                    // newest output column (tap 0)
                win[0] = (ox0 < W) ? Pair2<T>::load(gy + static_cast<long long>(ox0) * C) : make_float2(0.f, 0.f);
                const float2 xv = Pair2<T>::load(xr + static_cast<long long>(sx) * C);
#pragma unroll
                for (int l = 0; l < MAXW; ++l) {
                    acc[l].x = fmaf(xv.x, win[l].x, acc[l].x);
                    acc[l].y = fmaf(xv.y, win[l].y, acc[l].y);
                }
#pragma unroll
                for (int l = MAXW - 1; l > 0; --l) win[l] = win[l - 1];
            }
        }
#pragma unroll
        for (int l = 0; l < MAXW; ++l)
            if (l < kw) {
                float* dst = dweight + static_cast<long long>(ij * kw + l) * C + c;
                atomicAdd(dst, acc[l].x);
                atomicAdd(dst + 1, acc[l].y);
            }
        if (ij == 0 && dbias) {
            atomicAdd(dbias + c, bsum.x);
            atomicAdd(dbias + c + 1, bsum.y);
        }
    }
}

// The 3 x 3 x 3 kernel in bf16, staged like dwconv3d_tma_kernel: a CTA owns a column of
// 4 x 16 positions x 64 channels and marches along t; the x planes (with their halo) sit in a
// ring of 4 shared-memory slots and the dy planes in a ring of 2, each fetched by TMA one step
// ahead.  A lane owns a pair of channels, a warp one row of 16 positions: per kernel row it
// slides over 18 x words against the row's 16 dy words, all 27 x 2 sums in registers (packed
// fp32 FMAs).  The four warps reduce in shared memory; one vector atomic per four channels
// and tap goes to dweight.
constexpr int kWgTY = 4, kWgTX = 16, kWgXRing = 4, kWgYRing = 2;
constexpr int kWgXPlane = (kWgTY + 2) * (kWgTX + 2) * kCvCh * 2;        // 13824 bytes
constexpr int kWgYPlane = kWgTY * kWgTX * kCvCh * 2;                    // 8192 bytes
struct __align__(128) WgradSmem {
    unsigned char xp[kWgXRing][kWgXPlane];
    unsigned char yp[kWgYRing][kWgYPlane];
    float red[28][kCvCh];
    uint64_t xbar[kWgXRing], ybar[kWgYRing];
};

__global__ void __launch_bounds__(128)
dwconv3d_wgrad333_tma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_dy,
                             float* __restrict__ dweight, float* __restrict__ dbias, int Tn, int H, int W, int C,
                             int t_chunk) {
    extern __shared__ unsigned char raw_smem[];
    WgradSmem& s = *reinterpret_cast<WgradSmem*>((reinterpret_cast<uintptr_t>(raw_smem) + 127) & ~uintptr_t(127));
    const int tid = threadIdx.x, lane = tid & 31, yl = tid >> 5;
    const int c0 = blockIdx.x * kCvCh;
    const int tiles_x = (W + kWgTX - 1) / kWgTX;
    const int x0 = (blockIdx.y % tiles_x) * kWgTX, y0 = (blockIdx.y / tiles_x) * kWgTY;
    const int t_begin = blockIdx.z * t_chunk, t_end = min(Tn, t_begin + t_chunk);

    for (int i = tid; i < 28 * kCvCh; i += 128) (&s.red[0][0])[i] = 0.0f;
    if (tid == 0) {
        for (int i = 0; i < kWgXRing; ++i) mbar_init(smem_u32(&s.xbar[i]), 1);
        for (int i = 0; i < kWgYRing; ++i) mbar_init(smem_u32(&s.ybar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // x plane n is frame t_begin - 1 + n (slot n % 4); dy plane m is frame t_begin + m (slot m % 2)
    auto issue_x = [&](int n) {
        const int slot = n % kWgXRing;
        mbar_expect_tx(smem_u32(&s.xbar[slot]), kWgXPlane);
        tma_load_4d(smem_u32(s.xp[slot]), &map_x, smem_u32(&s.xbar[slot]), c0, x0 - 1, y0 - 1, t_begin - 1 + n);
    };
    auto issue_y = [&](int m) {
        const int slot = m % kWgYRing;
        mbar_expect_tx(smem_u32(&s.ybar[slot]), kWgYPlane);
        tma_load_4d(smem_u32(s.yp[slot]), &map_dy, smem_u32(&s.ybar[slot]), c0, x0, y0, t_begin + m);
    };
    if (tid == 0) {
        for (int n = 0; n < 3; ++n) issue_x(n);
        issue_y(0);
    }

    float2 acc[27];
#pragma unroll
    for (int k = 0; k < 27; ++k) acc[k] = make_float2(0.f, 0.f);
    float2 bsum = make_float2(0.f, 0.f);
    bool ok = true;

    for (int t = t_begin; t < t_end && ok; ++t) {
        const int m = t - t_begin;                                      // dy plane; x planes m, m+1, m+2
        if (tid == 0 && t + 1 < t_end) {                                // slots last read by step t-1
            issue_x(m + 3);
            issue_y(m + 1);
        }
        for (int n = (m == 0 ? 0 : m + 2); n <= m + 2; ++n)
            if (!mbar_wait(smem_u32(&s.xbar[n % kWgXRing]), (n / kWgXRing) & 1)) ok = false;
        if (!mbar_wait(smem_u32(&s.ybar[m % kWgYRing]), (m / kWgYRing) & 1)) ok = false;
        if (!ok) atomicExch(&g_timeout_flag, 11);
        ok = __syncthreads_and(ok);                                     // all threads stop together or not at all
        if (!ok) break;
        // this warp's row of dy: 16 words per lane
        const uint32_t* gy = reinterpret_cast<const uint32_t*>(s.yp[m % kWgYRing]) + (yl * kWgTX) * (kCvCh / 2) + lane;
        float2 g[kWgTX];
#pragma unroll
        for (int ox = 0; ox < kWgTX; ++ox) {
            const uint32_t r = gy[ox * (kCvCh / 2)];
            g[ox] = make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
            bsum.x += g[ox].x;
            bsum.y += g[ox].y;
        }
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t* plane = reinterpret_cast<const uint32_t*>(s.xp[(m + i) % kWgXRing]);
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const uint32_t* xrow = plane + ((yl + j) * (kWgTX + 2)) * (kCvCh / 2) + lane;
#pragma unroll
                for (int sx = 0; sx < kWgTX + 2; ++sx) {                // input column x0 - 1 + sx
                    const uint32_t r = xrow[sx * (kCvCh / 2)];
                    const float x_lo = __uint_as_float(r << 16), x_hi = __uint_as_float(r & 0xffff0000u);
#pragma unroll
                    for (int l = 0; l < 3; ++l) {
                        const int ox = sx - l;                          // output column that tap l pairs with it
                        if (ox < 0 || ox >= kWgTX) continue;
                        float2& a = acc[(i * 3 + j) * 3 + l];
                        fma2(a.x, a.y, x_lo, x_hi, g[ox].x, g[ox].y);
                    }
                }
            }
        }
        __syncthreads();                                                // the oldest x slot and this dy slot are free
    }
    // rows of the tile beyond the grid carry zeros (TMA fill), so no masking is needed
#pragma unroll
    for (int k = 0; k < 27; ++k) {
        atomicAdd(&s.red[k][lane * 2], acc[k].x);
        atomicAdd(&s.red[k][lane * 2 + 1], acc[k].y);
    }
    atomicAdd(&s.red[27][lane * 2], bsum.x);
    atomicAdd(&s.red[27][lane * 2 + 1], bsum.y);
    __syncthreads();
    for (int i = tid; i < 28 * (kCvCh / 4); i += 128) {
        const int k = i / (kCvCh / 4), q = (i % (kCvCh / 4)) * 4;
        float* dst = k < 27 ? dweight + static_cast<long long>(k) * C + c0 + q : (dbias ? dbias + c0 + q : nullptr);
        if (dst)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(s.red[k][q]), "f"(s.red[k][q + 1]),
                         "f"(s.red[k][q + 2]), "f"(s.red[k][q + 3])
                         : "memory");
    }
}

// The 3 x 3 x 3 forward in bf16 with the same lane mapping as the weight-gradient kernel above:
// a lane owns a pair of channels and holds their 27 x 2 weights in registers, a warp one row of
// 16 outputs; per kernel row it slides over 18 x words (one 4-byte shared-memory read each, 128
// contiguous bytes per warp) and feeds 16 x 2 sums by packed fp32 FMAs.  Against the general
// staged kernel (8 channels x 4 outputs per thread, weights re-read from shared memory per
// kernel row) this is a third fewer instructions per output.
#ifndef DSA3D_CONV3_RING
#define DSA3D_CONV3_RING 4
#endif
constexpr int kCv3Ring = DSA3D_CONV3_RING;          // resident planes: 3 in use + the ones on their way
struct __align__(128) Conv333Smem {
    unsigned char xp[kCv3Ring][kWgXPlane];
    uint64_t xbar[kCv3Ring];
};

__global__ void __launch_bounds__(128)
dwconv3d_333_tma_kernel(const __grid_constant__ CUtensorMap map_x, const float* __restrict__ weight,
                        const float* __restrict__ bias, __nv_bfloat16* __restrict__ y, int Tn, int H, int W, int C,
                        int t_chunk, int ct, int chh, int cw) {
    extern __shared__ unsigned char raw_smem[];
    Conv333Smem& s = *reinterpret_cast<Conv333Smem*>((reinterpret_cast<uintptr_t>(raw_smem) + 127) & ~uintptr_t(127));
    const int tid = threadIdx.x, lane = tid & 31, yl = tid >> 5;
    const int c0 = blockIdx.x * kCvCh;
    const int tiles_x = (W + kWgTX - 1) / kWgTX;
    const int x0 = (blockIdx.y % tiles_x) * kWgTX, y0 = (blockIdx.y / tiles_x) * kWgTY;
    const int t_begin = blockIdx.z * t_chunk, t_end = min(Tn, t_begin + t_chunk);
    if (tid == 0) {
        for (int i = 0; i < kCv3Ring; ++i) mbar_init(smem_u32(&s.xbar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // x plane n is frame t_begin - ct + n (slot n % ring); output t reads planes m .. m+2, m = t - t_begin
    auto issue_x = [&](int n) {
        const int slot = n % kCv3Ring;
        mbar_expect_tx(smem_u32(&s.xbar[slot]), kWgXPlane);
        tma_load_4d(smem_u32(s.xp[slot]), &map_x, smem_u32(&s.xbar[slot]), c0, x0 - cw, y0 - chh, t_begin - ct + n);
    };
    const int planes = t_end - t_begin + 2;                           // planes this CTA ever needs
    if (tid == 0)
        for (int n = 0; n < kCv3Ring - 1 && n < planes; ++n) issue_x(n);

    float2 wv[27];
#pragma unroll
    for (int k = 0; k < 27; ++k)
        wv[k] = __ldg(reinterpret_cast<const float2*>(weight + static_cast<long long>(k) * C + c0 + lane * 2));
    const float2 bv = bias ? __ldg(reinterpret_cast<const float2*>(bias + c0 + lane * 2)) : make_float2(0.f, 0.f);
    const int oy = y0 + yl;
    bool ok = true;

    for (int t = t_begin; t < t_end && ok; ++t) {
        const int m = t - t_begin;
        if (tid == 0 && m + kCv3Ring - 1 < planes) issue_x(m + kCv3Ring - 1);   // its slot was last read by output t-1
        for (int n = (m == 0 ? 0 : m + 2); n <= m + 2; ++n)
            if (!mbar_wait(smem_u32(&s.xbar[n % kCv3Ring]), (n / kCv3Ring) & 1)) ok = false;
        if (!ok) atomicExch(&g_timeout_flag, 12);
        ok = __syncthreads_and(ok);                                     // all threads stop together or not at all
        if (!ok) break;
        float2 acc[kWgTX];
#pragma unroll
        for (int ox = 0; ox < kWgTX; ++ox) acc[ox] = bv;
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const uint32_t* plane = reinterpret_cast<const uint32_t*>(s.xp[(m + i) % kCv3Ring]);
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const uint32_t* xrow = plane + ((yl + j) * (kWgTX + 2)) * (kCvCh / 2) + lane;
#pragma unroll
                for (int sx = 0; sx < kWgTX + 2; ++sx) {                // input column x0 - cw + sx
                    const uint32_t r = xrow[sx * (kCvCh / 2)];
                    const float x_lo = __uint_as_float(r << 16), x_hi = __uint_as_float(r & 0xffff0000u);
#pragma unroll
                    for (int l = 0; l < 3; ++l) {
                        const int ox = sx - l;                          // output that tap l maps this input to
                        if (ox < 0 || ox >= kWgTX) continue;
                        const float2 w2 = wv[(i * 3 + j) * 3 + l];
#ifdef DSA3D_CONV3_PLAIN_FMA
                        acc[ox].x = fmaf(x_lo, w2.x, acc[ox].x);
                        acc[ox].y = fmaf(x_hi, w2.y, acc[ox].y);
#else
                        fma2(acc[ox].x, acc[ox].y, x_lo, x_hi, w2.x, w2.y);
#endif
                    }
                }
            }
        }
        if (oy < H) {
            __nv_bfloat16* dst = y + ((static_cast<long long>(t) * H + oy) * W + x0) * C + c0 + lane * 2;
#pragma unroll
            for (int ox = 0; ox < kWgTX; ++ox)
                if (x0 + ox < W) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(acc[ox].x, acc[ox].y);
                    *reinterpret_cast<__nv_bfloat162*>(dst + static_cast<long long>(ox) * C) = h;
                }
        }
        __syncthreads();                                                // the oldest plane may now be overwritten
    }
}

bool try_dwconv_333(const void* x, const float* weight, const float* bias, void* y, int T, int H, int W, int C,
                    const int centre[3], cudaStream_t st, cudaError_t* err) {
    *err = cudaSuccess;
    const int tiles = ((W + kWgTX - 1) / kWgTX) * ((H + kWgTY - 1) / kWgTY);
    CUtensorMap map;
    if (tiles > 65535 || !make_map_activations(&map, x, T, H, W, C, kWgTX + 2, kWgTY + 2)) return false;
    int splits = 1;
    const long long columns = static_cast<long long>(C / kCvCh) * tiles;
    while (columns * splits < 148 * 8 && T / (splits * 2) >= 12) splits *= 2;
    const int t_chunk = (T + splits - 1) / splits;
    const size_t smem = sizeof(Conv333Smem) + 128;
    *err = cudaFuncSetAttribute(dwconv3d_333_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (*err != cudaSuccess) return true;
    const dim3 grid(C / kCvCh, tiles, (T + t_chunk - 1) / t_chunk);
    dwconv3d_333_tma_kernel<<<grid, 128, smem, st>>>(map, weight, bias, static_cast<__nv_bfloat16*>(y), T, H, W, C, t_chunk,
                                                     centre[0], centre[1], centre[2]);
    *err = cudaGetLastError();
    return true;
}

template <typename T>
cudaError_t launch_wgrad(const void* x, const void* dy, float* dweight, float* dbias, int Tn, int H, int W, int C,
                         const int kernel[3], cudaStream_t st) {
    const long long rows = static_cast<long long>(Tn) * H;
    if (std::is_same<T, __nv_bfloat16>::value && kernel[0] == 3 && kernel[1] == 3 && kernel[2] == 3 && C % kCvCh == 0 &&
        !std::getenv("DSA3D_WGRAD_PLAIN")) {
        const int tiles = ((W + kWgTX - 1) / kWgTX) * ((H + kWgTY - 1) / kWgTY);
        CUtensorMap map_x, map_dy;
        if (tiles <= 65535 && make_map_activations(&map_x, x, Tn, H, W, C, kWgTX + 2, kWgTY + 2) &&
            make_map_activations(&map_dy, dy, Tn, H, W, C, kWgTX, kWgTY)) {
            int splits = 1;                                  // as in the forward: fill the GPU, keep chunks long
            const long long columns = static_cast<long long>(C / kCvCh) * tiles;
            while (columns * splits < 148 * 8 && Tn / (splits * 2) >= 12) splits *= 2;
            const int t_chunk = (Tn + splits - 1) / splits;
            const size_t smem = sizeof(WgradSmem) + 128;
            cudaError_t e = cudaFuncSetAttribute(dwconv3d_wgrad333_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 static_cast<int>(smem));
            if (e != cudaSuccess) return e;
            const dim3 grid(C / kCvCh, tiles, (Tn + t_chunk - 1) / t_chunk);
            dwconv3d_wgrad333_tma_kernel<<<grid, 128, smem, st>>>(map_x, map_dy, dweight, dbias, Tn, H, W, C, t_chunk);
            return cudaGetLastError();
        }
    }
    const long long chunks = (rows + kWgradRows - 1) / kWgradRows;
    if (chunks > 65535) return cudaErrorInvalidConfiguration;
    int warps = kernel[0] * kernel[1];
    if (warps > 32) warps = 32;
    const dim3 grid((C + 63) / 64, static_cast<unsigned>(chunks));
    const T* xp = static_cast<const T*>(x);
    const T* gp = static_cast<const T*>(dy);
#define DSA3D_WGRAD_CASE(KW) \
    case KW: dwconv3d_wgrad_kernel<T, KW><<<grid, warps * 32, 0, st>>>(xp, gp, dweight, dbias, Tn, H, W, C, kernel[0], kernel[1], KW); break;
    switch (kernel[2]) {
        DSA3D_WGRAD_CASE(1)
        DSA3D_WGRAD_CASE(3)
        DSA3D_WGRAD_CASE(5)
        DSA3D_WGRAD_CASE(7)
        default: dwconv3d_wgrad_kernel<T, 0><<<grid, warps * 32, 0, st>>>(xp, gp, dweight, dbias, Tn, H, W, C, kernel[0], kernel[1], kernel[2]);
    }
#undef DSA3D_WGRAD_CASE
    return cudaGetLastError();
}

// src [rows, cols] (row pitch lds) -> dstT [cols, rows] bf16 (row pitch ldt, a multiple of 8); when
// `dst` is given also the untransposed bf16 copy (row pitch ldd, a multiple of 8: whole words are
// written, the padding columns included), and when `colsum` is given the fp32 column sums of src
// (one atomic per column and block).  A block owns a 64-column strip of up to kTrRowsPerBlock
// rows and walks it in 64 x 64 tiles through shared memory; a thread moves pairs: two
// neighbouring columns on the way in, two neighbouring rows on the way out, so every warp
// access is 128 contiguous bytes (256 for fp32 sources).
constexpr int kTrRowsPerBlock = 1024;
template <typename S> struct SrcPair;
template <> struct SrcPair<float> {
    static __device__ __forceinline__ float2 load(const float* p, bool vec, bool second) {
        if (vec) return __ldg(reinterpret_cast<const float2*>(p));
        return make_float2(__ldg(p), second ? __ldg(p + 1) : 0.0f);
    }
};
template <> struct SrcPair<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(const __nv_bfloat16* p, bool vec, bool second) {
        if (vec) {
            const uint32_t r = __ldg(reinterpret_cast<const uint32_t*>(p));
            return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
        }
        return make_float2(__bfloat162float(p[0]), second ? __bfloat162float(p[1]) : 0.0f);
    }
};

template <typename S>
__global__ void __launch_bounds__(256)
transpose_to_bf16_kernel(const S* __restrict__ src, long long lds, long long rows, int cols,
                         __nv_bfloat16* __restrict__ dstT, long long ldt, __nv_bfloat16* __restrict__ dst, long long ldd,
                         float* __restrict__ colsum) {
    __shared__ uint32_t tile[64][33];                                // [row][column pair]
    __shared__ float sums[8][64];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 pairs x 8 phases
    const int c0 = blockIdx.x * 64;
    const long long rb = static_cast<long long>(blockIdx.y) * kTrRowsPerBlock;
    const long long re = rb + kTrRowsPerBlock < rows ? rb + kTrRowsPerBlock : rows;
    const int c = c0 + 2 * tx;
    const bool in0 = c < cols, in1 = c + 1 < cols;
    // a pair is one aligned vector when the row pitch keeps pairs aligned and both columns exist
    const bool vec = in1 && (lds & 1) == 0 && (reinterpret_cast<uintptr_t>(src) & (2 * sizeof(S) - 1)) == 0;
    float s0 = 0.0f, s1 = 0.0f;
    for (long long t0 = rb; t0 < re; t0 += 64) {
#pragma unroll
        for (int r = ty; r < 64; r += 8) {
            const long long row = t0 + r;
            float2 v = make_float2(0.0f, 0.0f);
            if (row < re && in0) v = SrcPair<S>::load(src + row * lds + c, vec, in1);
            s0 += v.x;
            s1 += v.y;
            const __nv_bfloat162 h = __floats2bfloat162_rn(v.x, v.y);
            const uint32_t word = *reinterpret_cast<const uint32_t*>(&h);
            if (dstT) tile[r][tx] = word;
            if (dst && row < re && c < ldd) *reinterpret_cast<uint32_t*>(dst + row * ldd + c) = word;
        }
        if (!dstT) continue;                                         // copy and column sums only (uniform)
        __syncthreads();
        // rows 2tx, 2tx+1 of column pair j: one word per column, each the two rows' values
        const long long row = t0 + 2 * tx;
#pragma unroll
        for (int j = ty; j < 32; j += 8) {
            const uint32_t a = tile[2 * tx][j], b = tile[2 * tx + 1][j];
            const int cc = c0 + 2 * j;
            if (row < re) {                                          // row + 1 < ldt: the pitch is even
                if (cc < cols)
                    *reinterpret_cast<uint32_t*>(dstT + static_cast<long long>(cc) * ldt + row) = __byte_perm(a, b, 0x5410);
                if (cc + 1 < cols)
                    *reinterpret_cast<uint32_t*>(dstT + static_cast<long long>(cc + 1) * ldt + row) = __byte_perm(a, b, 0x7632);
            }
        }
        __syncthreads();
    }
    if (colsum) {
        sums[ty][2 * tx] = s0;
        sums[ty][2 * tx + 1] = s1;
        __syncthreads();
        if (threadIdx.x < 64 && c0 + threadIdx.x < cols) {
            float t = 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) t += sums[k][threadIdx.x];
            atomicAdd(colsum + c0 + threadIdx.x, t);
        }
    }
}

// fp32 [rows, cols] -> bf16 copy (row pitch ldd) plus fp32 column sums, for cols a multiple of 4:
// a thread owns four neighbouring columns and walks down kCvtRows rows, so a block reads whole
// rows front to back (one contiguous stream per block) and issues one atomic per column.
constexpr int kCvtRows = 512;
__global__ void __launch_bounds__(1024)
convert_rows_bf16_kernel(const float* __restrict__ src, long long rows, int cols, __nv_bfloat16* __restrict__ dst,
                         long long ldd, float* __restrict__ colsum) {
    const long long rb = static_cast<long long>(blockIdx.x) * kCvtRows;
    const long long re = rb + kCvtRows < rows ? rb + kCvtRows : rows;
    for (int c = threadIdx.x * 4; c < cols; c += blockDim.x * 4) {
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* sp = src + rb * cols + c;
        __nv_bfloat16* dp = dst + rb * ldd + c;
#pragma unroll 4
        for (long long r = rb; r < re; ++r, sp += cols, dp += ldd) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(sp));
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
            *reinterpret_cast<uint2*>(dp) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo),
                                                       *reinterpret_cast<const uint32_t*>(&hi));
        }
        if (colsum) {
            atomicAdd(colsum + c, sum.x);
            atomicAdd(colsum + c + 1, sum.y);
            atomicAdd(colsum + c + 2, sum.z);
            atomicAdd(colsum + c + 3, sum.w);
        }
    }
}

// fp32 storage: plain loops, one thread per output element.
__global__ void __launch_bounds__(256)
linear_du_f32_kernel(const float* __restrict__ g, const float* __restrict__ w, float* __restrict__ du, long long M, int C,
                     int O) {
    const long long id = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (id >= M * C) return;
    const long long n = id / C;
    const int c = static_cast<int>(id - n * C);
    float acc = 0.0f;
    for (int o = 0; o < O; ++o) acc = fmaf(__ldg(g + n * O + o), __ldg(w + static_cast<long long>(o) * C + c), acc);
    du[id] = acc;
}

__global__ void __launch_bounds__(256)
linear_dw_f32_kernel(const float* __restrict__ g, const float* __restrict__ u, float* __restrict__ dw,
                     float* __restrict__ dbias, long long M, int C, int O) {
    const long long id = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (id >= static_cast<long long>(O) * C) return;
    const int o = static_cast<int>(id / C), c = static_cast<int>(id % C);
    float acc = 0.0f, bs = 0.0f;
    for (long long n = 0; n < M; ++n) {
        const float gv = __ldg(g + n * O + o);
        acc = fmaf(gv, __ldg(u + n * C + c), acc);
        bs += gv;
    }
    if (dw) dw[id] = acc;
    if (dbias && c == 0) dbias[o] = bs;
}

long long round_up8(long long v) { return (v + 7) / 8 * 8; }
size_t round_up256(size_t v) { return (v + 255) / 256 * 256; }
constexpr long long kLinearSlabTokens = 262144;          // tokens per pass of the linear layer's backward

struct LinearBackwardPlan {
    long long slab, ld_o;
    size_t off_wt, off_g, total;
};
LinearBackwardPlan linear_backward_plan(long long tokens, int C, int O) {
    LinearBackwardPlan p;
    p.slab = tokens < kLinearSlabTokens ? tokens : kLinearSlabTokens;
    p.ld_o = round_up8(O);
    size_t at = 0;
    p.off_wt = at; at += round_up256(static_cast<size_t>(C) * p.ld_o * 2);          // w^T  [C, O]
    p.off_g = at;  at += round_up256(static_cast<size_t>(p.slab) * p.ld_o * 2);     // doffsets in bf16 [slab, O]
    p.total = at;
    return p;
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

namespace {
// Test aid (dsa3d_test_wait_timeout): one thread waits, with a small poll limit, on an mbarrier
// that nothing ever arrives at, then gives up the way every bounded wait of the library does:
// it raises the timeout flag (value 99) and returns.  No TMA, no TMEM, nothing to drain.
__global__ void wait_timeout_probe_kernel(unsigned polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_limit(smem_u32(&bar), 0u, polls)) atomicExch(&g_timeout_flag, 99);
    }
}
}  // namespace

int* dsa3d::timeout_flag_device_address() {
    void* p = nullptr;
    return cudaGetSymbolAddress(&p, g_timeout_flag) == cudaSuccess ? static_cast<int*>(p) : nullptr;
}

namespace {

int cuda_failed(cudaError_t e) { return dsa3d::note_cuda_error(e); }

// y = cross-correlation of x with weight; tap (i, j, l) reads the input at displacement
// (i - centre[0], j - centre[1], l - centre[2]).
int conv_entry(const void* x, const float* weight, const float* bias, int T, int H, int W, int C, const int kernel[3],
               const int centre[3], void* y, int dtype, void* stream) {
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
        if (try_dwconv_tma(x, weight, bias, y, T, H, W, C, kernel, centre, st, &te))
            return te == cudaSuccess ? DSA3D_OK : cuda_failed(te);
    }
    if (dtype == DSA3D_BF16)
        launch_dwconv<__nv_bfloat16>(x, weight, bias, y, T, H, W, C, kernel, centre, static_cast<unsigned>(blocks), st);
    else
        launch_dwconv<float>(x, weight, bias, y, T, H, W, C, kernel, centre, static_cast<unsigned>(blocks), st);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

}  // namespace

extern "C" {

int dsa3d_dwconv3d_forward(const void* x, const float* weight, const float* bias, int T, int H, int W, int C,
                           const int kernel[3], void* y, int dtype, void* stream) {
    if (!kernel) return DSA3D_ERR_NULL_POINTER;
    const int centre[3] = {kernel[0] / 2, kernel[1] / 2, kernel[2] / 2};
    return conv_entry(x, weight, bias, T, H, W, C, kernel, centre, y, dtype, stream);
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
        bool unsupported = false;
        e = launch_pair_gemm(u, static_cast<unsigned long long>(C), w, static_cast<unsigned long long>(C), bias, offsets,
                             tokens, O, C, kGemmStoreF32, 1, sms, st, &unsupported);
        if (unsupported) return DSA3D_ERR_UNSUPPORTED;
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

size_t dsa3d_dwconv3d_backward_workspace_bytes(int C, const int kernel[3]) {
    if (!kernel || C < 1 || kernel[0] < 1 || kernel[1] < 1 || kernel[2] < 1) return 0;
    return round_up256(static_cast<size_t>(kernel[0]) * kernel[1] * kernel[2] * C * sizeof(float));
}

int dsa3d_dwconv3d_backward(const void* x, const float* weight, const void* dy, int T, int H, int W, int C,
                            const int kernel[3], void* dx, float* dweight, float* dbias, void* workspace,
                            size_t workspace_bytes, int dtype, void* stream) {
    if (!dy || !kernel || (dx && (!weight || !workspace)) || (dweight && !x) || (dbias && !dweight))
        return DSA3D_ERR_NULL_POINTER;
    if (T < 1 || H < 1 || W < 1 || C < 8 || C % 8) return DSA3D_ERR_BAD_SHAPE;
    if (kernel[0] < 1 || kernel[1] < 1 || kernel[2] < 1 || kernel[2] > kConvMaxKw || kernel[0] > 15 || kernel[1] > 15)
        return DSA3D_ERR_BAD_SHAPE;
    if (dtype != DSA3D_F32 && dtype != DSA3D_BF16) return DSA3D_ERR_UNSUPPORTED;
    if (!aligned16(dy) || (x && !aligned16(x)) || (dx && !aligned16(dx)) || (dweight && !aligned16(dweight)) ||
        (dbias && !aligned16(dbias)) || (weight && !aligned16(weight)) || (workspace && !aligned16(workspace)))
        return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int taps = kernel[0] * kernel[1] * kernel[2];
    if (dx) {
        if (workspace_bytes < dsa3d_dwconv3d_backward_workspace_bytes(C, kernel)) return DSA3D_ERR_WORKSPACE;
        float* wf = static_cast<float*>(workspace);
        const long long n = static_cast<long long>(taps) * C;
        flip_weight_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(weight, wf, taps, C);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_failed(e);
        // flipped tap i' = kt-1-i reads dy at displacement i' - (kt-1-kt/2)
        const int centre[3] = {kernel[0] - 1 - kernel[0] / 2, kernel[1] - 1 - kernel[1] / 2, kernel[2] - 1 - kernel[2] / 2};
        const int rc = conv_entry(dy, wf, nullptr, T, H, W, C, kernel, centre, dx, dtype, stream);
        if (rc != DSA3D_OK) return rc;
    }
    if (dweight) {
        cudaError_t e = cudaMemsetAsync(dweight, 0, static_cast<size_t>(taps) * C * sizeof(float), st);
        if (e != cudaSuccess) return cuda_failed(e);
        if (dbias) {
            e = cudaMemsetAsync(dbias, 0, static_cast<size_t>(C) * sizeof(float), st);
            if (e != cudaSuccess) return cuda_failed(e);
        }
        e = dtype == DSA3D_BF16 ? launch_wgrad<__nv_bfloat16>(x, dy, dweight, dbias, T, H, W, C, kernel, st)
                                : launch_wgrad<float>(x, dy, dweight, dbias, T, H, W, C, kernel, st);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return DSA3D_OK;
}

size_t dsa3d_offsets_linear_backward_workspace_bytes(long long tokens, int C, int O, int dtype) {
    if (tokens < 1 || C < 1 || O < 1 || dtype != DSA3D_BF16) return 0;
    return linear_backward_plan(tokens, C, O).total;
}

int dsa3d_offsets_linear_backward(const void* u, const void* w, const float* doffsets, long long tokens, int C, int O,
                                  void* du, float* dw, float* dbias, void* workspace, size_t workspace_bytes, int dtype,
                                  void* stream) {
    if (!doffsets || (du && !w) || (dw && !u)) return DSA3D_ERR_NULL_POINTER;
    if (tokens < 1 || C < 8 || C % 8 || O < 1 || tokens > 0x7fffffffLL) return DSA3D_ERR_BAD_SHAPE;
    if (dtype != DSA3D_F32 && dtype != DSA3D_BF16) return DSA3D_ERR_UNSUPPORTED;
    if (!aligned16(doffsets) || (u && !aligned16(u)) || (w && !aligned16(w)) || (du && !aligned16(du)) ||
        (dw && !aligned16(dw)) || (workspace && !aligned16(workspace)))
        return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (dtype == DSA3D_F32) {
        if (du) {
            const long long blocks = (tokens * C + 255) / 256;
            if (blocks > 0x7fffffffLL) return DSA3D_ERR_BAD_SHAPE;
            linear_du_f32_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(
                doffsets, static_cast<const float*>(w), static_cast<float*>(du), tokens, C, O);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_failed(e);
        }
        if (dw || dbias) {
            if (!u) return DSA3D_ERR_NULL_POINTER;
            const long long blocks = (static_cast<long long>(O) * C + 255) / 256;
            linear_dw_f32_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(doffsets, static_cast<const float*>(u), dw,
                                                                                 dbias, tokens, C, O);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_failed(e);
        }
        return DSA3D_OK;
    }
    if (!du && !dw && !dbias) return DSA3D_OK;
    if (!workspace) return DSA3D_ERR_NULL_POINTER;
    const LinearBackwardPlan plan = linear_backward_plan(tokens, C, O);
    if (workspace_bytes < plan.total) return DSA3D_ERR_WORKSPACE;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return cuda_failed(e);
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return cuda_failed(e);
    if (sms < 2) return DSA3D_ERR_UNSUPPORTED;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    __nv_bfloat16* wt = reinterpret_cast<__nv_bfloat16*>(ws + plan.off_wt);
    __nv_bfloat16* g = reinterpret_cast<__nv_bfloat16*>(ws + plan.off_g);
    const __nv_bfloat16* ub = static_cast<const __nv_bfloat16*>(u);
    if (dw && (e = cudaMemsetAsync(dw, 0, static_cast<size_t>(O) * C * sizeof(float), st)) != cudaSuccess) return cuda_failed(e);
    if (dbias && (e = cudaMemsetAsync(dbias, 0, static_cast<size_t>(O) * sizeof(float), st)) != cudaSuccess) return cuda_failed(e);
    if (du) {                                                        // w [O, C] -> w^T [C, O]
        const dim3 grid((C + 63) / 64, static_cast<unsigned>((O + kTrRowsPerBlock - 1) / kTrRowsPerBlock));
        transpose_to_bf16_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w), C, O, C, wt,
                                                                      plan.ld_o, nullptr, 0, nullptr);
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_failed(e);
    }
    bool unsupported = false;
    for (long long s0 = 0; s0 < tokens; s0 += plan.slab) {
        const long long ns = tokens - s0 < plan.slab ? tokens - s0 : plan.slab;
        const unsigned row_blocks = static_cast<unsigned>((ns + kTrRowsPerBlock - 1) / kTrRowsPerBlock);
        if (O % 4 == 0) {   // doffsets slab -> bf16 copy and column sums
            int threads = ((O / 4 + 31) / 32) * 32;
            if (threads > 1024) threads = 1024;
            convert_rows_bf16_kernel<<<static_cast<unsigned>((ns + kCvtRows - 1) / kCvtRows), threads, 0, st>>>(
                doffsets + s0 * O, ns, O, g, plan.ld_o, dbias);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_failed(e);
        } else {            // rows that do not start on a 16-byte boundary: the pairwise kernel
            const dim3 grid((O + 63) / 64, row_blocks);
            transpose_to_bf16_kernel<float><<<grid, 256, 0, st>>>(doffsets + s0 * O, O, ns, O, nullptr, 0, g, plan.ld_o,
                                                                  dbias);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_failed(e);
        }
        if (du) {                                                    // du[slab] = g . (w^T)^T
            e = launch_pair_gemm(g, static_cast<unsigned long long>(plan.ld_o), wt, static_cast<unsigned long long>(plan.ld_o),
                                 nullptr, static_cast<__nv_bfloat16*>(du) + s0 * C, ns, C, O, kGemmStoreBf16, 1, sms, st,
                                 &unsupported);
            if (unsupported) return DSA3D_ERR_UNSUPPORTED;
            if (e != cudaSuccess) return cuda_failed(e);
        }
        if (dw) {       // dw += g^T . u over this slab's tokens: both operands have the contraction index as rows
            const long long tiles = ((O + 2 * BM - 1) / (2 * BM)) * static_cast<long long>((C + kMaxBN - 1) / kMaxBN);
            const long long kblocks = (ns + BK - 1) / BK;
            long long ksplits = (2LL * (sms / 2) + tiles - 1) / tiles;        // about two waves of work units
            if (ksplits > kblocks) ksplits = kblocks;
            if (ksplits < 1) ksplits = 1;
            e = launch_pair_gemm(g, static_cast<unsigned long long>(plan.ld_o), ub + s0 * C, static_cast<unsigned long long>(C),
                                 nullptr, dw, O, C, static_cast<int>(ns), kGemmAddF32, static_cast<int>(ksplits), sms, st,
                                 &unsupported, true);
            if (unsupported) return DSA3D_ERR_UNSUPPORTED;
            if (e != cudaSuccess) return cuda_failed(e);
        }
    }
    return DSA3D_OK;
}

int dsa3d_device_timeout_flag(void) {
    int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_timeout_flag, sizeof(int)) != cudaSuccess) return -1;
    return flag;
}

int dsa3d_check_device_timeout(void) {
    const int flag = dsa3d_device_timeout_flag();
    if (flag < 0) return cuda_failed(cudaGetLastError());
    return flag == 0 ? DSA3D_OK : DSA3D_ERR_DEVICE_TIMEOUT;
}

int dsa3d_clear_device_timeout(void) {
    const int zero = 0;
    const cudaError_t e = cudaMemcpyToSymbol(g_timeout_flag, &zero, sizeof(int));
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

int dsa3d_test_wait_timeout(unsigned polls, void* stream) {
    if (polls < 1 || polls > (1u << 20)) return DSA3D_ERR_BAD_SHAPE;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(polls);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

}  // extern "C"
