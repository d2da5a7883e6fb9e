// Fixed-window backward (all offsets zero), the three weighted sums of rows as tile kernels:
//     dQ_i = sum_p ck_{i,p} K_{i+b(p)},   dK_j = sum_p ck_{j-b(p),p} q_{j-b(p)},   dV_j = sum_p cv_{j-b(p),p} dO_{j-b(p)}
// (ck = scale dS, cv = alpha: the two coefficients per sample that fixed_window_backward_query_kernel leaves;
// the chain rule of the Formulation with every sample on a grid position).  Taken per output row these are
// P row gathers each - 27 rows of 256 bytes through the L2-to-SM port per (row, head), which is what bounds
// the per-row kernels.  Taken per tile of 4 x 4 x 8 output rows the rows needed form the tile's halo region
// (6 x 6 x 10 for a 3 x 3 x 3 window), shared by the tile's 128 outputs: the region arrives once by TMA and
// every row in it is read from shared memory, widened once, and added to each of the up to kw outputs of its
// x-row whose window holds it - the forward's output phase with other weights.
//
// One persistent CTA per SM walks (tile, head) items; an item is three sweeps - dQ over the K region, dK over
// the q region, dV over the dO region - and the sweeps of the CTA's items form one stream: while sweep g runs
// from one region buffer the TMA load of sweep g + 1 fills the other and the coefficients of sweep g + 1 are
// on their way into registers (stored as that sweep's weight table afterwards).  bf16, 64 or 128 channels,
// windows (3,3,3) and (2,2,2); everything else keeps the per-row kernels.  The wait on a load is bounded and
// raises the library's timeout flag.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kTgTT = 4, kTgTY = 4, kTgTX = 8;            // outputs per tile
constexpr int kTgThreads = 256;                           // 16 half-warps = the 4 x 4 x-rows of the tile

template <int D, int KT, int KH, int KW>
struct TgShape {
    static constexpr int RT = kTgTT + KT - 1, RY = kTgTY + KH - 1, RX = kTgTX + KW - 1;
    static constexpr int X_BYTES = (RT * RY * RX * D * 2 + 1023) / 1024 * 1024;
    static constexpr int W_FLOATS = 16 * KT * KH * kTgTX * KW;            // [x-row][kernel row (u, v)][output][w]
    static constexpr int W_PER_THREAD = (W_FLOATS + kTgThreads - 1) / kTgThreads;
    // origin of the region below the tile: a gather (dQ) reaches k/2 back, a scatter seen from its target
    // (dK, dV) reaches k - 1 - k/2 back
    static constexpr int FT = KT / 2, FY = KH / 2, FX = KW / 2;
    static constexpr int BT = KT - 1 - KT / 2, BY = KH - 1 - KH / 2, BX = KW - 1 - KW / 2;
    static_assert((kTgTX * KW) % 4 == 0, "a kernel row's weights are read as 16-byte pieces");
};

template <int D, int KT, int KH, int KW>
struct __align__(1024) TgSmem {
    using S = TgShape<D, KT, KH, KW>;
    unsigned char x[2][S::X_BYTES];               // region rows, unswizzled: [t][y][x][D channels]
    float w[2][S::W_FLOATS];
    uint64_t bar[2];
    uint32_t abort;
};

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kTgThreads, 1)
fixed_window_tile_grad_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                              const __grid_constant__ CUtensorMap map_do, const float2* __restrict__ coef,
                              __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                              int T, int H, int W, int heads, int tiles_x, int tiles_y, int total, int* timeout_flag) {
    using S = TgShape<D, KT, KH, KW>;
    constexpr int RY = S::RY, RX = S::RX, P = KT * KH * KW;
    constexpr int CPL = D / 16;                                   // channels per lane of a half-warp
    extern __shared__ unsigned char raw[];
    TgSmem<D, KT, KH, KW>& s =
        *reinterpret_cast<TgSmem<D, KT, KH, KW>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(smem_u32(&s.bar[0]), 1);
        mbar_init(smem_u32(&s.bar[1]), 1);
        s.abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile uint32_t* abort_flag = &s.abort;

    const int tiles_per_head = total / heads;
    const int my_items = static_cast<int>(blockIdx.x) < total
                             ? (total - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;
    const int sweeps = 3 * my_items;
    // sweep g of this CTA: item g / 3, and which sum (0: dQ over K, 1: dK over q, 2: dV over dO)
    auto locate = [&](int g, int& m, int& t0, int& y0, int& x0) {
        const int item = static_cast<int>(blockIdx.x) + (g / 3) * static_cast<int>(gridDim.x);
        m = item / tiles_per_head;
        int tile = item - m * tiles_per_head;
        x0 = (tile % tiles_x) * kTgTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kTgTY;
        t0 = (tile / tiles_y) * kTgTT;
    };
    auto load_region = [&](int g) {                               // thread 0 only
        int m, t0, y0, x0;
        locate(g, m, t0, y0, x0);
        const int which = g % 3;
        const uint32_t bar = smem_u32(&s.bar[g & 1]);
        mbar_expect_tx(bar, static_cast<uint32_t>(S::RT * RY * RX) * D * 2u);
        const CUtensorMap* map = which == 0 ? &map_k : which == 1 ? &map_q : &map_do;
        const int ot = which == 0 ? S::FT : S::BT, oy = which == 0 ? S::FY : S::BY, ox = which == 0 ? S::FX : S::BX;
        tma_load_5d(smem_u32(s.x[g & 1]), map, bar, 0, m, x0 - ox, y0 - oy, t0 - ot);
    };
    // This thread's entries of sweep g's weight table, from the coefficient array.  The loads are unconditional
    // (a query that does not exist reads entry 0 and is zeroed when the table is stored, `dead` remembers which):
    // a load under a condition has to be merged with the old register value as soon as it is issued, and the
    // thread would wait out the latency of each load in turn.
    auto fetch_weights = [&](int g, float (&wv)[S::W_PER_THREAD], uint32_t& dead) {
        int m, t0, y0, x0;
        locate(g, m, t0, y0, x0);
        const int which = g % 3;
        const float* cf = reinterpret_cast<const float*>(coef) + (which == 2 ? 1 : 0);
        dead = 0u;
#pragma unroll
        for (int i = 0; i < S::W_PER_THREAD; ++i) {
            const int e = tid + i * kTgThreads;
            const int ww = e % KW, qx = (e / KW) % kTgTX, uv = (e / (KW * kTgTX)) % (KT * KH), hw = e / (KW * kTgTX * KT * KH);
            const int u = uv / KH, vv = uv - u * KH, lt = hw >> 2, ly = hw & 3;
            int qt, qy, qxx, p;
            if (which == 0) {                                     // output = the query itself, cell (u, vv, ww)
                qt = t0 + lt; qy = y0 + ly; qxx = x0 + qx;
                p = (u * KH + vv) * KW + ww;
            } else {                                              // output = a key; the query at region offset (u, vv, ww) of it
                qt = t0 + lt - S::BT + u; qy = y0 + ly - S::BY + vv; qxx = x0 + qx - S::BX + ww;
                p = ((KT - 1 - u) * KH + (KH - 1 - vv)) * KW + (KW - 1 - ww);
            }
            const bool exists = e < S::W_FLOATS && qt >= 0 && qt < T && qy >= 0 && qy < H && qxx >= 0 && qxx < W;
            const long long at = exists ? ((((static_cast<long long>(qt) * H + qy) * W + qxx) * heads + m) * P + p) : 0;
            wv[i] = __ldg(cf + 2 * at);
            if (!exists) dead |= 1u << i;
        }
    };
    auto store_weights = [&](int g, const float (&wv)[S::W_PER_THREAD], uint32_t dead) {
#pragma unroll
        for (int i = 0; i < S::W_PER_THREAD; ++i) {
            const int e = tid + i * kTgThreads;
            if (e < S::W_FLOATS) s.w[g & 1][e] = ((dead >> i) & 1u) ? 0.0f : wv[i];
        }
    };

    float wv[S::W_PER_THREAD];
    uint32_t dead = 0u;
    static_assert(S::W_PER_THREAD <= 32, "one bit per entry");
    if (sweeps > 0) {
        if (tid == 0) load_region(0);
        fetch_weights(0, wv, dead);
        store_weights(0, wv, dead);
    }
    __syncthreads();

    for (int g = 0; g < sweeps; ++g) {
        if (g + 1 < sweeps) {
            if (tid == 0 && !*abort_flag) load_region(g + 1);     // its buffer was read by sweep g - 1, which has ended
            fetch_weights(g + 1, wv, dead);
        }
        // ---- the region of sweep g has arrived (every thread polls: all of them read it)
        if (!*abort_flag && !mbar_wait(smem_u32(&s.bar[g & 1]), static_cast<uint32_t>((g >> 1) & 1))) {
            atomicExch(timeout_flag, 41);
            *abort_flag = 1u;
        }
        // ---- a half-warp per x-row of 8 outputs, CPL channels per lane
        {
            const int hw = tid >> 4, hl = tid & 15;
            const int lt = hw >> 2, ly = hw & 3;
            float acc[kTgTX][CPL];
#pragma unroll
            for (int qx = 0; qx < kTgTX; ++qx)
#pragma unroll
                for (int e = 0; e < CPL; ++e) acc[qx][e] = 0.0f;
            const float* wrow = s.w[g & 1] + hw * (KT * KH * kTgTX * KW);
            const unsigned char* xbuf = s.x[g & 1];
#pragma unroll 1
            for (int uv = 0; uv < KT * KH; ++uv) {
                const int u = uv / KH, vv = uv - u * KH;
                float wq[kTgTX * KW];                             // the 8 outputs' KW weights of this kernel row
#pragma unroll
                for (int i = 0; i < kTgTX * KW; i += 4) {
                    const float4 w4 = *reinterpret_cast<const float4*>(wrow + uv * (kTgTX * KW) + i);
                    wq[i] = w4.x; wq[i + 1] = w4.y; wq[i + 2] = w4.z; wq[i + 3] = w4.w;
                }
                const unsigned char* xrow = xbuf + (((lt + u) * RY + ly + vv) * RX) * (D * 2) + hl * (CPL * 2);
#pragma unroll
                for (int xx = 0; xx < RX; ++xx) {
                    uint32_t words[CPL / 2];
                    if constexpr (CPL == 8) {
                        const uint4 row = *reinterpret_cast<const uint4*>(xrow + xx * (D * 2));
                        words[0] = row.x; words[1] = row.y; words[2] = row.z; words[3] = row.w;
                    } else {
                        const uint2 row = *reinterpret_cast<const uint2*>(xrow + xx * (D * 2));
                        words[0] = row.x; words[1] = row.y;
                    }
                    float f[CPL];
#pragma unroll
                    for (int i = 0; i < CPL / 2; ++i) {
                        f[2 * i] = __uint_as_float(words[i] << 16);
                        f[2 * i + 1] = __uint_as_float(words[i] & 0xffff0000u);
                    }
#pragma unroll
                    for (int ww = 0; ww < KW; ++ww) {
                        const int qx = xx - ww;                   // the output whose cell ww is region position xx
                        if (qx < 0 || qx >= kTgTX) continue;
#pragma unroll
                        for (int e = 0; e < CPL; e += 2)
                            fma2(acc[qx][e], acc[qx][e + 1], wq[qx * KW + ww], wq[qx * KW + ww], f[e], f[e + 1]);
                    }
                }
            }
            int m, t0, y0, x0;
            locate(g, m, t0, y0, x0);
            const int which = g % 3;
            __nv_bfloat16* out = which == 0 ? dq : which == 1 ? dk : dv;
            const int t = t0 + lt, y = y0 + ly;
            if (!*abort_flag && t < T && y < H) {
#pragma unroll
                for (int qx = 0; qx < kTgTX; ++qx) {
                    const int x = x0 + qx;
                    if (x >= W) continue;
                    const long long n = (static_cast<long long>(t) * H + y) * W + x;
                    uint32_t o[CPL / 2];
#pragma unroll
                    for (int i = 0; i < CPL / 2; ++i) {
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[qx][2 * i], acc[qx][2 * i + 1]);
                        o[i] = *reinterpret_cast<const uint32_t*>(&h2);
                    }
                    __nv_bfloat16* dst = out + (n * heads + m) * D + hl * CPL;
                    if constexpr (CPL == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                    else *reinterpret_cast<uint2*>(dst) = make_uint2(o[0], o[1]);
                }
            }
        }
        if (g + 1 < sweeps) store_weights(g + 1, wv, dead);      // the other table: read last by sweep g - 1
        __syncthreads();                                         // sweep g's region and table are free
    }
    // gave up: a load may still be on its way into this CTA's shared memory
    if (*abort_flag && tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_wait_limit(smem_u32(&s.bar[i]), 0u, 1u << 16);
            mbar_wait_limit(smem_u32(&s.bar[i]), 1u, 1u << 16);
        }
    }
}

template <int D, int KT, int KH, int KW>
cudaError_t launch_tile_grad(const void* q, const void* k, const void* dout, const float2* coef, void* dq, void* dk, void* dv,
                             const Problem& pr, int* flag, cudaStream_t stream, bool* unsupported) {
    using S = TgShape<D, KT, KH, KW>;
    const unsigned long long d = static_cast<unsigned long long>(pr.d), hd = static_cast<unsigned long long>(pr.heads);
    const unsigned long long dims[5] = {d, hd, static_cast<unsigned long long>(pr.W), static_cast<unsigned long long>(pr.H),
                                        static_cast<unsigned long long>(pr.T)};
    const unsigned long long strides[4] = {d * 2, hd * d * 2, static_cast<unsigned long long>(pr.W) * hd * d * 2,
                                           static_cast<unsigned long long>(pr.H) * pr.W * hd * d * 2};
    const unsigned box[5] = {static_cast<unsigned>(pr.d), 1, static_cast<unsigned>(S::RX), static_cast<unsigned>(S::RY),
                             static_cast<unsigned>(S::RT)};
    CUtensorMap mk, mq, mdo;
    if (!encode_tensor_map_bf16(&mk, k, 5, dims, strides, box, false) || !encode_tensor_map_bf16(&mq, q, 5, dims, strides, box, false) ||
        !encode_tensor_map_bf16(&mdo, dout, 5, dims, strides, box, false)) {
        *unsupported = true;
        return cudaSuccess;
    }
    const int tiles_x = (pr.W + kTgTX - 1) / kTgTX, tiles_y = (pr.H + kTgTY - 1) / kTgTY, tiles_t = (pr.T + kTgTT - 1) / kTgTT;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    if (total * 3 >= (1LL << 31)) {                                // the kernel counts sweeps in 32 bits
        *unsupported = true;
        return cudaSuccess;
    }
    const size_t smem = sizeof(TgSmem<D, KT, KH, KW>) + 1024;
    auto kern = fixed_window_tile_grad_kernel<D, KT, KH, KW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kTgThreads, smem, stream>>>(mk, mq, mdo, coef, static_cast<__nv_bfloat16*>(dq), static_cast<__nv_bfloat16*>(dk),
                                             static_cast<__nv_bfloat16*>(dv), pr.T, pr.H, pr.W, pr.heads, tiles_x, tiles_y,
                                             static_cast<int>(total), flag);
    return cudaGetLastError();
}

}  // namespace

bool fixed_window_tile_grad_covers(const Problem& pr, bool bf16) {
    if (!bf16 || (pr.d != 128 && pr.d != 64)) return false;
    return (pr.kt == 3 && pr.kh == 3 && pr.kw == 3) || (pr.kt == 2 && pr.kh == 2 && pr.kw == 2);
}

bool try_fixed_window_tile_grad(const void* q, const void* k, const void* dout, const float2* coef, void* dq, void* dk, void* dv,
                                const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (!fixed_window_tile_grad_covers(pr, true)) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    const bool w333 = pr.kt == 3;
    if (pr.d == 128)
        *err = w333 ? launch_tile_grad<128, 3, 3, 3>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_tile_grad<128, 2, 2, 2>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    else
        *err = w333 ? launch_tile_grad<64, 3, 3, 3>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_tile_grad<64, 2, 2, 2>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    return !unsupported;
}

}  // namespace dsa3d
