// Fixed-window forward (all offsets zero: the local-attention variant of the ablation on the
// effect of offsets) as dense tile attention.  With zero offsets sample p of a query sits
// exactly on the grid position query + b(p), so the logits of a tile of queries are entries
// of the dense product  Q_tile . K_region^T  over the tile's halo region, and the window is a
// mask on that score tile.
//
// Persistent CTAs, a work item = (tile of 4 x 4 x 8 queries, head); bf16, 64 or 128 channels:
//   1. TMA 5-D boxes bring the tile's Q rows (128 x 128), the K rows of the region
//      (tile + kt-1, kh-1, kw-1 halo; zero rows outside the grid, which is exactly the
//      zero-padded key of a sample outside the grid) in the 128-byte-swizzled K-major layout,
//      and the V rows of the region unswizzled.
//   2. One thread issues tcgen05.mma (M = 128, N <= 192 per instruction, K = 16 x 8) into
//      fp32 accumulators in TMEM: S[query, region position].
//   3. Warp w owns the queries of tile plane w.  It copies the score columns of the kt region
//      planes its queries can see from TMEM to shared memory (tcgen05.ld, one column per
//      bank), each thread picks the P entries of its window, does the softmax in registers
//      (dead samples keep logit 0, as in the general kernel) and leaves normalised weights
//      in shared memory.
//   4. All 8 warps form the output: a half-warp per x-row of 8 queries, 8 channels per lane;
//      each V row of the x-row's reach is read from shared memory and widened once and added
//      into every query whose window holds it, with fp32 weights (no rounding of the weights).
// Waits on mbarriers are bounded and raise the library's timeout flag.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kFwTT = 4, kFwTY = 4, kFwTX = 8, kFwQ = kFwTT * kFwTY * kFwTX;   // 128 queries per tile
constexpr int kFwThreads = 256;
constexpr int kFwMaxRows = 368;                   // region rows held per K half / V (multiple of 16)

template <int D>
struct __align__(1024) FwSmem {
    unsigned char q[D / 64][kFwQ * 128];          // 64-channel halves, 128-byte rows; later score staging + weights
    unsigned char k[D / 64][kFwMaxRows * 128];    // 64-channel halves
    unsigned char v[kFwMaxRows * D * 2];          // full rows
    unsigned char w[D == 64 ? 16 * 1024 : 16];    // 64 channels: the softmax weights (the Q buffer is only 16 KB)
    uint64_t bar_q, bar_k, bar_v, bar_mma;
    uint32_t tmem_base;
    uint32_t abort;                               // set by the issuing thread when one of its waits ran out
};

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kFwThreads, 1)
fixed_window_forward_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                            const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ out,
                            float* __restrict__ lse, int T, int H, int W, int heads, int tiles_x, int tiles_y,
                            long long total, int* timeout_flag) {
    constexpr int P = KT * KH * KW;
    constexpr int NH = D / 64;                                    // 64-channel halves of a row
    constexpr int CPL = D / 16;                                   // channels per lane in the output phase
    constexpr int RT = kFwTT + KT - 1, RY = kFwTY + KH - 1, RX = kFwTX + KW - 1;
    constexpr int PS = RY * RX;                                   // rows of one region plane
    constexpr int R = RT * PS;                                    // region rows
    constexpr int RP = (R + 15) / 16 * 16;                        // padded to the MMA's N granularity
    constexpr int N1 = RP <= 192 ? RP : 192, N2 = RP - N1;
    constexpr int kChunks = (PS + 31) / 32;                       // 32-column pieces of a region plane
    static_assert(RP <= kFwMaxRows && N2 <= 256 && P <= 32, "shape not covered");
    static_assert((RT - 1) * PS + kChunks * 32 <= 512, "staged columns must stay inside the TMEM allocation");
    static_assert(16 * KT * KH * kFwTX * KW * 4 <= 16 * 1024, "the weights must fit their 16 KB");

    extern __shared__ unsigned char raw[];
    FwSmem<D>& s = *reinterpret_cast<FwSmem<D>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(smem_u32(&s.bar_q), 1);
        mbar_init(smem_u32(&s.bar_k), 1);
        mbar_init(smem_u32(&s.bar_v), 1);
        mbar_init(smem_u32(&s.bar_mma), 1);
        s.abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;
    bool ok = true;

    // Work item -> (head, tile origin); tiles of one head are neighbours in the launch order.
    const long long tiles_per_head = total / heads;
    auto locate = [&](long long item, int& m, int& t0, int& y0, int& x0) {
        m = static_cast<int>(item / tiles_per_head);
        int tile = static_cast<int>(item - m * tiles_per_head);
        x0 = (tile % tiles_x) * kFwTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kFwTY;
        t0 = (tile / tiles_y) * kFwTT;
    };
    auto load_q = [&](int m, int t0, int y0, int x0) {
        mbar_expect_tx(smem_u32(&s.bar_q), static_cast<uint32_t>(NH) * kFwQ * 128u);
        for (int h = 0; h < NH; ++h) tma_load_5d(smem_u32(s.q[h]), &map_q, smem_u32(&s.bar_q), h * 64, m, x0, y0, t0);
    };
    auto load_k = [&](int m, int t0, int y0, int x0) {
        mbar_expect_tx(smem_u32(&s.bar_k), static_cast<uint32_t>(NH) * R * 128u);
        for (int h = 0; h < NH; ++h)
            tma_load_5d(smem_u32(s.k[h]), &map_k, smem_u32(&s.bar_k), h * 64, m, x0 - KW / 2, y0 - KH / 2, t0 - KT / 2);
    };
    auto load_v = [&](int m, int t0, int y0, int x0) {
        mbar_expect_tx(smem_u32(&s.bar_v), static_cast<uint32_t>(R) * D * 2u);
        tma_load_5d(smem_u32(s.v), &map_v, smem_u32(&s.bar_v), 0, m, x0 - KW / 2, y0 - KH / 2, t0 - KT / 2);
    };

    float* stage = reinterpret_cast<float*>(s.q[0]);              // [32 columns][128 threads]: lower half of the Q buffer
    // softmax weights: the second 16 KB of the Q buffer (128 channels) or their own array (64)
    float* wts = reinterpret_cast<float*>(NH == 1 ? s.w : s.q[0] + 16 * 1024);

    if (tid == 0 && static_cast<long long>(blockIdx.x) < total) {
        int m, t0, y0, x0;
        locate(blockIdx.x, m, t0, y0, x0);
        load_q(m, t0, y0, x0);
        load_k(m, t0, y0, x0);
        load_v(m, t0, y0, x0);
    }

    uint32_t parity = 0;
    for (long long item = blockIdx.x; item < total && ok; item += gridDim.x, parity ^= 1u) {
        int m, t0, y0, x0;
        locate(item, m, t0, y0, x0);
        const long long next = item + gridDim.x;

        // ---- 2. score tile, then the next tile's K into the buffer the MMAs have finished with
        if (tid == 0) {
            if (mbar_wait(smem_u32(&s.bar_q), parity) && mbar_wait(smem_u32(&s.bar_k), parity)) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kFwQ >> 4) << 24);
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const uint64_t da = smem_desc(smem_u32(s.q[h]));
                    const uint64_t db1 = smem_desc(smem_u32(s.k[h]));
                    const uint64_t db2 = smem_desc(smem_u32(s.k[h]) + N1 * 128);       // N1 rows = a multiple of 8
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {                                   // 16 channels = 32 bytes per step
                        umma_bf16(tmem, da + 2 * kk, db1 + 2 * kk, idesc_base | (static_cast<uint32_t>(N1 >> 3) << 17),
                                  (h | kk) ? 1u : 0u);
                        if (N2 > 0)
                            umma_bf16(tmem + N1, da + 2 * kk, db2 + 2 * kk,
                                      idesc_base | (static_cast<uint32_t>(N2 >> 3) << 17), (h | kk) ? 1u : 0u);
                    }
                }
            } else {
                atomicExch(timeout_flag, 5);
                *reinterpret_cast<volatile uint32_t*>(&s.abort) = 1u;
            }
            umma_commit(smem_u32(&s.bar_mma));
            if (next < total && mbar_wait(smem_u32(&s.bar_mma), parity)) {
                int m2, t2, y2, x2;
                locate(next, m2, t2, y2, x2);
                load_k(m2, t2, y2, x2);
            }
        }

        // ---- 3. window extraction and softmax: warps 0-3, one query per thread
        if (warp < 4) {
            if (!mbar_wait(smem_u32(&s.bar_mma), parity)) {
                if (lane == 0) atomicExch(timeout_flag, 6);
                ok = false;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            __syncwarp();
            const int r = tid;                                    // query row = TMEM lane
            const int lt = warp, ly = lane >> 3, lx = lane & 7;   // box order of the Q load: x fastest, then y, then t
            float sc[P];
            if (ok) {
#pragma unroll
                for (int u = 0; u < KT; ++u) {
                    // columns of region plane lt + u, 32 at a time, through shared memory:
                    // stage[column][thread], one bank per thread
#pragma unroll
                    for (int ch = 0; ch < kChunks; ++ch) {
                        uint32_t regs[32];
                        tmem_load_32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + (lt + u) * PS + ch * 32, regs);
#pragma unroll
                        for (int i = 0; i < 32; ++i) stage[i * kFwQ + r] = __uint_as_float(regs[i]);
                        __syncwarp();
#pragma unroll
                        for (int vv = 0; vv < KH; ++vv)
#pragma unroll
                            for (int ww = 0; ww < KW; ++ww) {
                                const int idx = (ly + vv) * RX + lx + ww - ch * 32;
                                if (idx >= 0 && idx < 32) sc[(u * KH + vv) * KW + ww] = stage[idx * kFwQ + r];
                            }
                        __syncwarp();
                    }
                }
                const float lscale = rsqrtf(static_cast<float>(D)) * kLog2e;
                float mx = -INFINITY;
#pragma unroll
                for (int p = 0; p < P; ++p) { sc[p] *= lscale; mx = fmaxf(mx, sc[p]); }
                float sum = 0.0f;
#pragma unroll
                for (int p = 0; p < P; ++p) { sc[p] = exp2f(sc[p] - mx); sum += sc[p]; }
                const float inv = 1.0f / sum;
                // weights of an x-row of 8 queries together: [row of the tile][u, v][lx][w]
                float* wrow = wts + (warp * kFwTY + ly) * (KT * KH * kFwTX * KW) + lx * KW;
#pragma unroll
                for (int uv = 0; uv < KT * KH; ++uv)
#pragma unroll
                    for (int ww = 0; ww < KW; ++ww) wrow[uv * (kFwTX * KW) + ww] = sc[uv * KW + ww] * inv;
                const int t = t0 + lt, y = y0 + ly, x = x0 + lx;
                if (t < T && y < H && x < W) {
                    const long long n = (static_cast<long long>(t) * H + y) * W + x;
                    lse[n * heads + m] = (mx + log2f(sum)) * kLn2;
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
        if (!mbar_wait(smem_u32(&s.bar_v), parity)) {
            if (tid == 0) atomicExch(timeout_flag, 7);
            ok = false;
        }
        if (*reinterpret_cast<volatile uint32_t*>(&s.abort)) ok = false;
        ok = __syncthreads_and(ok);       // every thread takes the same decision to go on or to stop

        // ---- 4. output: a half-warp per x-row of 8 queries, 8 channels per lane.  Neighbouring
        //         queries share most of their window, so each V row of the x-row's reach is read
        //         and widened once and added into every query whose window holds it.
        {
            const int hw = tid >> 4, hl = tid & 15;               // 16 half-warps = the 4 x 4 x-rows of the tile
            const int lt = hw >> 2, ly = hw & 3;
            float acc[kFwTX][CPL];
#pragma unroll
            for (int qx = 0; qx < kFwTX; ++qx)
#pragma unroll
                for (int e = 0; e < CPL; ++e) acc[qx][e] = 0.0f;
            const float* wrow = wts + hw * (KT * KH * kFwTX * KW);
#pragma unroll 1
            for (int uv = 0; uv < KT * KH; ++uv) {
                const int u = uv / KH, vv = uv - u * KH;
                float wq[kFwTX * KW];                             // the 8 queries' KW weights of this kernel row
#pragma unroll
                for (int i = 0; i < kFwTX * KW; i += 4) {
                    const float4 w4 = *reinterpret_cast<const float4*>(wrow + uv * (kFwTX * KW) + i);
                    wq[i] = w4.x; wq[i + 1] = w4.y; wq[i + 2] = w4.z; wq[i + 3] = w4.w;
                }
                const unsigned char* vrow = s.v + (((lt + u) * RY + ly + vv) * RX) * (D * 2) + hl * (CPL * 2);
#pragma unroll
                for (int xx = 0; xx < RX; ++xx) {
                    uint32_t words[CPL / 2];
                    if constexpr (CPL == 8) {
                        const uint4 row = *reinterpret_cast<const uint4*>(vrow + xx * (D * 2));
                        words[0] = row.x; words[1] = row.y; words[2] = row.z; words[3] = row.w;
                    } else {
                        const uint2 row = *reinterpret_cast<const uint2*>(vrow + xx * (D * 2));
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
                        const int qx = xx - ww;                   // the query whose window cell ww is position xx
                        if (qx < 0 || qx >= kFwTX) continue;
#pragma unroll
                        for (int e = 0; e < CPL; e += 2)                  // two FMAs per instruction
                            fma2(acc[qx][e], acc[qx][e + 1], wq[qx * KW + ww], wq[qx * KW + ww], f[e], f[e + 1]);
                    }
                }
            }
            const int t = t0 + lt, y = y0 + ly;
            if (ok && t < T && y < H) {
#pragma unroll
                for (int qx = 0; qx < kFwTX; ++qx) {
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
        __syncthreads();              // the weights (Q buffer) and V have been read: refill both
        if (tid == 0 && next < total) {
            int m2, t2, y2, x2;
            locate(next, m2, t2, y2, x2);
            load_q(m2, t2, y2, x2);
            load_v(m2, t2, y2, x2);
        }
    }
    if (!ok && tid == 0) {            // stopped early: give loads still in flight a bounded time to land
        mbar_wait(smem_u32(&s.bar_k), parity);
        mbar_wait(smem_u32(&s.bar_q), parity);
        mbar_wait(smem_u32(&s.bar_v), parity);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
}

bool make_maps(const void* q, const void* k, const void* v, const Problem& pr, int kt, int kh, int kw, CUtensorMap* mq,
               CUtensorMap* mk, CUtensorMap* mv) {
    const unsigned long long d = static_cast<unsigned long long>(pr.d), hd = static_cast<unsigned long long>(pr.heads);
    const unsigned long long dims[5] = {d, hd, static_cast<unsigned long long>(pr.W), static_cast<unsigned long long>(pr.H),
                                        static_cast<unsigned long long>(pr.T)};
    const unsigned long long strides[4] = {d * 2, hd * d * 2, static_cast<unsigned long long>(pr.W) * hd * d * 2,
                                           static_cast<unsigned long long>(pr.H) * pr.W * hd * d * 2};
    const unsigned box_q[5] = {64, 1, kFwTX, kFwTY, kFwTT};
    const unsigned box_k[5] = {64, 1, static_cast<unsigned>(kFwTX + kw - 1), static_cast<unsigned>(kFwTY + kh - 1),
                               static_cast<unsigned>(kFwTT + kt - 1)};
    const unsigned box_v[5] = {static_cast<unsigned>(pr.d), 1, box_k[2], box_k[3], box_k[4]};
    return encode_tensor_map_bf16(mq, q, 5, dims, strides, box_q, true) &&
           encode_tensor_map_bf16(mk, k, 5, dims, strides, box_k, true) &&
           encode_tensor_map_bf16(mv, v, 5, dims, strides, box_v, false);
}

template <int D, int KT, int KH, int KW>
cudaError_t launch(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, void* out, float* lse,
                   const Problem& pr, int* flag, cudaStream_t stream) {
    const int tiles_x = (pr.W + kFwTX - 1) / kFwTX, tiles_y = (pr.H + kFwTY - 1) / kFwTY,
              tiles_t = (pr.T + kFwTT - 1) / kFwTT;
    const size_t smem = sizeof(FwSmem<D>) + 1024;
    auto kern = fixed_window_forward_kernel<D, KT, KH, KW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kFwThreads, smem, stream>>>(mq, mk, mv, static_cast<__nv_bfloat16*>(out), lse, pr.T, pr.H, pr.W, pr.heads,
                                             tiles_x, tiles_y, total, flag);
    return cudaGetLastError();
}

}  // namespace

bool try_fixed_window_forward(const void* q, const void* k, const void* v, void* out, float* lse, const Problem& pr,
                              cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (pr.d != 128 && pr.d != 64) return false;
    const bool w333 = pr.kt == 3 && pr.kh == 3 && pr.kw == 3, w222 = pr.kt == 2 && pr.kh == 2 && pr.kw == 2;
    if (!w333 && !w222) return false;
    const long long tiles = static_cast<long long>((pr.W + kFwTX - 1) / kFwTX) * ((pr.H + kFwTY - 1) / kFwTY) *
                            ((pr.T + kFwTT - 1) / kFwTT);
    if (tiles > 0x7fffffffLL) return false;
    int* flag = timeout_flag_device_address();
    CUtensorMap mq, mk, mv;
    if (!flag || !make_maps(q, k, v, pr, pr.kt, pr.kh, pr.kw, &mq, &mk, &mv)) return false;
    if (pr.d == 128)
        *err = w333 ? launch<128, 3, 3, 3>(mq, mk, mv, out, lse, pr, flag, stream)
                    : launch<128, 2, 2, 2>(mq, mk, mv, out, lse, pr, flag, stream);
    else
        *err = w333 ? launch<64, 3, 3, 3>(mq, mk, mv, out, lse, pr, flag, stream)
                    : launch<64, 2, 2, 2>(mq, mk, mv, out, lse, pr, flag, stream);
    return true;
}

}  // namespace dsa3d
