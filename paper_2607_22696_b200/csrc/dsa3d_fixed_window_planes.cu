// Fixed-window forward for windows larger than 3 x 3 x 3 (the paper's own (3,7,7) of its
// zero-offset ablation, and (3,5,5)) as dense tile attention with BOTH contractions on the
// tensor cores, one region plane at a time.
//
// With zero offsets sample p of a query sits on the grid position query + b(p), so the logits
// of a tile of queries are entries of  Q_tile . K_region^T  and the output is  P . V_region
// with P the softmax weights placed at their region positions (zero elsewhere).  The halo
// region of a 4 x 4 x 8 query tile holds (4+kt-1)(4+kh-1)(8+kw-1) key rows - 840 for (3,7,7) -
// more than TMEM columns or shared memory take at once, so the tile walks the region's kt+3
// planes (along t) twice:
//
//   pass 1, plane by plane:  K plane by TMA (zero rows outside the grid = the zero-padded key of
//     a dead sample) -> S_plane = Q . K_plane^T by tcgen05.mma into one of two TMEM buffers ->
//     the two warps that share a TMEM quadrant copy the plane's score columns to shared memory,
//     every thread picks the window cells of its query that lie in this plane (static register
//     indices).  Two threads serve a query (the window's kernel rows are split between them).
//   softmax in registers; the pair of threads exchanges max and sum through shared memory; lse out.
//   pass 2, plane by plane:  V plane by TMA into the same ring of buffers; every thread writes its
//     query's row of P_plane into shared memory in the 128-byte-swizzled K-major layout, each
//     fp32 weight split into a bf16 head and a bf16 remainder (relative error of the pair 2^-17,
//     far inside the rounding of the output); two chains of tcgen05.mma (head and remainder, V as
//     an MN-major operand) accumulate  O += P_plane . V_plane  in TMEM.
//   epilogue: O from TMEM, one rounding to bf16, out.
//
// One thread issues every TMA load and every MMA.  Loads run two planes ahead through a ring of
// two plane buffers.  Every wait on an mbarrier is bounded; a wait that runs out raises the
// library's timeout flag and the CTA stops after draining its loads and freeing its TMEM.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kPlTT = 4, kPlTY = 4, kPlTX = 8, kPlQ = kPlTT * kPlTY * kPlTX;    // 128 queries per tile
constexpr int kPlThreads = 256;

template <int D, int KT, int KH, int KW>
struct PlaneShape {
    static constexpr int NH = D / 64;                               // 64-channel halves of a row
    static constexpr int RT = kPlTT + KT - 1, RY = kPlTY + KH - 1, RX = kPlTX + KW - 1;
    static constexpr int PS = RY * RX;                              // key rows of one region plane
    static constexpr int PSP = (PS + 15) / 16 * 16;                 // padded to the MMA granularity
    static constexpr int KB = (PSP + 63) / 64;                      // 64-column blocks of a P row
    static constexpr int PIECES = (PS + 31) / 32;                   // 32-column pieces of a score plane
    static constexpr int VH = (KH + 1) / 2;                         // kernel rows of the first thread of a pair
    static constexpr int SBUF = (PIECES * 32 + 31) / 32 * 32;       // TMEM columns set aside per score buffer
    static constexpr int S0 = D, S1 = D + SBUF;                     // TMEM: O at 0, two score buffers behind it
    static constexpr int P_BYTES = KB * kPlQ * 128;                 // one P matrix (head or remainder)
    static constexpr int STAGE_BYTES = PIECES * 32 * kPlQ * 4;      // a score plane as [column][query] floats
    static constexpr int WORK_BYTES = (2 * P_BYTES > STAGE_BYTES ? 2 * P_BYTES : STAGE_BYTES);
    static constexpr int SLOT_HALF = PSP * 128;                     // one 64-channel half of a plane buffer
    static_assert(PSP <= 256, "a region plane must fit one MMA (N <= 256)");
    static_assert(D + 2 * SBUF <= 512, "TMEM columns");
    static_assert(SLOT_HALF % 1024 == 0 || true, "");
};

template <int D, int KT, int KH, int KW>
struct __align__(1024) PlSmem {
    using S = PlaneShape<D, KT, KH, KW>;
    unsigned char q[S::NH][kPlQ * 128];                             // 64-channel halves, swizzled 128-byte rows
    unsigned char slot[2][S::NH][(S::SLOT_HALF + 1023) / 1024 * 1024];   // K or V plane, same image for both uses
    unsigned char work[(S::WORK_BYTES + 1023) / 1024 * 1024];       // score staging (pass 1), P head + remainder (pass 2)
    float pair_max[kPlThreads], pair_sum[kPlThreads];
    uint64_t bar_q, bar_full[2], bar_s[2], bar_pv;
    uint32_t tmem_base;
};

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kPlThreads, 1)
fixed_window_planes_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ out,
                           float* __restrict__ lse, int T, int H, int W, int heads, int tiles_x, int tiles_y,
                           long long total, int* timeout_flag) {
    using S = PlaneShape<D, KT, KH, KW>;
    constexpr int NH = S::NH, RT = S::RT, RX = S::RX, PS = S::PS, PSP = S::PSP, VH = S::VH;
    constexpr int JOBS = 2 * RT;                                      // plane loads per tile: RT of K, then RT of V
    extern __shared__ unsigned char raw[];
    PlSmem<D, KT, KH, KW>& s =
        *reinterpret_cast<PlSmem<D, KT, KH, KW>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lt = warp & 3, half = warp >> 2;                        // query plane of the tile; which thread of the pair
    const int ly = lane >> 3, lx = lane & 7;                          // box order of the Q load: x fastest, then y, then t
    const int r = lt * 32 + lane;                                     // query row of the tile = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(lt * 32) << 16;

    if (tid == 0) {
        mbar_init(smem_u32(&s.bar_q), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&s.bar_full[i]), 1); mbar_init(smem_u32(&s.bar_s[i]), 1); }
        mbar_init(smem_u32(&s.bar_pv), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // rows PS .. PSP-1 of the plane buffers are never written by a load: they must read as zero
    // (as V rows they are multiplied by the zero columns of P; anything non-finite would spoil O)
    if constexpr (PSP > PS) {
        for (int i = tid; i < 2 * NH * (PSP - PS) * 8; i += kPlThreads) {
            const int chunk = i & 7, row = PS + (i >> 3) % (PSP - PS), which = (i >> 3) / (PSP - PS);
            *reinterpret_cast<uint4*>(&s.slot[which / NH][which % NH][row * 128 + chunk * 16]) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    const long long tiles_per_head = total / heads;
    auto locate = [&](long long item, int& m, int& t0, int& y0, int& x0) {
        m = static_cast<int>(item / tiles_per_head);
        int tile = static_cast<int>(item - m * tiles_per_head);
        x0 = (tile % tiles_x) * kPlTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kPlTY;
        t0 = (tile / tiles_y) * kPlTT;
    };
    // plane load number g of this CTA: tile g / JOBS, K plane (g % JOBS) or V plane (g % JOBS - RT)
    auto issue_load = [&](long long g) {
        const long long item = blockIdx.x + (g / JOBS) * static_cast<long long>(gridDim.x);
        if (item >= total) return;
        const int j = static_cast<int>(g % JOBS), sl = static_cast<int>(g & 1);
        int m, t0, y0, x0;
        locate(item, m, t0, y0, x0);
        const uint32_t bar = smem_u32(&s.bar_full[sl]);
        mbar_expect_tx(bar, static_cast<uint32_t>(NH) * PS * 128u);
        const CUtensorMap* map = j < RT ? &map_k : &map_v;
        for (int h = 0; h < NH; ++h)
            tma_load_5d(smem_u32(s.slot[sl][h]), map, bar, h * 64, m, x0 - KW / 2, y0 - KH / 2, t0 - KT / 2 + j % RT);
    };
    auto issue_q = [&](long long item) {
        if (item >= total) return;
        int m, t0, y0, x0;
        locate(item, m, t0, y0, x0);
        mbar_expect_tx(smem_u32(&s.bar_q), static_cast<uint32_t>(NH) * kPlQ * 128u);
        for (int h = 0; h < NH; ++h) tma_load_5d(smem_u32(s.q[h]), &map_q, smem_u32(&s.bar_q), h * 64, m, x0, y0, t0);
    };
    auto full_wait = [&](long long g) { return mbar_wait(smem_u32(&s.bar_full[g & 1]), static_cast<uint32_t>((g >> 1) & 1)); };

    constexpr uint32_t idesc_common = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kPlQ >> 4) << 24);
    // score plane number sp (counted over the CTA's life) -> TMEM buffer sp & 1
    auto issue_scores = [&](long long g, long long sp, bool first_of_tile, uint32_t q_parity) {
        bool ready = full_wait(g);
        if (ready && first_of_tile) ready = mbar_wait(smem_u32(&s.bar_q), q_parity);
        if (ready) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d_tmem = tmem + ((sp & 1) ? S::S1 : S::S0);
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                const uint64_t da = smem_desc(smem_u32(s.q[h])), db = smem_desc(smem_u32(s.slot[g & 1][h]));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc_common | (static_cast<uint32_t>(PSP >> 3) << 17),
                              (h | kk) ? 1u : 0u);
            }
        } else {
            atomicExch(timeout_flag, 13);
        }
        umma_commit(smem_u32(&s.bar_s[sp & 1]));                      // arrives at once if nothing was issued
        return ready;
    };

    if (tid == 0 && static_cast<long long>(blockIdx.x) < total) {
        issue_q(blockIdx.x);
        issue_load(0);
        issue_load(1);
    }

    float* stage = reinterpret_cast<float*>(s.work);                 // [column][query]
    unsigned char* p_head = s.work;
    unsigned char* p_rest = s.work + S::P_BYTES;
    const float lscale = rsqrtf(static_cast<float>(D)) * kLog2e;
    bool ok = true;
    long long it = 0;
    for (long long item = blockIdx.x; item < total && ok; item += gridDim.x, ++it) {
        int m, t0, y0, x0;
        locate(item, m, t0, y0, x0);
        const long long g0 = it * JOBS, sp0 = it * RT;
        float sc[KT][VH][KW];
#pragma unroll
        for (int u = 0; u < KT; ++u)
#pragma unroll
            for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                for (int ww = 0; ww < KW; ++ww) sc[u][vi][ww] = -INFINITY;

        // ------------------------------------------------------------ pass 1: scores, plane by plane
        if (tid == 0 && !issue_scores(g0, sp0, true, static_cast<uint32_t>(it & 1))) ok = false;
        for (int pl = 0; pl < RT; ++pl) {
            const long long g = g0 + pl, sp = sp0 + pl;
            if (tid == 0 && pl + 1 < RT && ok && !issue_scores(g + 1, sp + 1, false, 0u)) ok = false;
            if (!mbar_wait(smem_u32(&s.bar_s[sp & 1]), static_cast<uint32_t>((sp >> 1) & 1))) {
                if (lane == 0) atomicExch(timeout_flag, 14);
                ok = false;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (tid == 0 && ok) {                                     // this plane's buffer is free: two planes ahead
                issue_load(g + 2);
                if (pl == RT - 1) issue_q(item + gridDim.x);          // all score MMAs of the tile have read Q
            }
            const int u_rt = pl - lt;                                 // the kernel plane this region plane is to the warp's queries
            if (u_rt >= 0 && u_rt < KT) {
                const uint32_t sbuf = tmem + lane_base + ((sp & 1) ? S::S1 : S::S0);
                for (int piece = half; piece < S::PIECES; piece += 2) {
                    uint32_t regs[32];
                    tmem_load_32(sbuf + piece * 32, regs);
#pragma unroll
                    for (int i = 0; i < 32; ++i) stage[(piece * 32 + i) * kPlQ + r] = __uint_as_float(regs[i]);
                }
                named_barrier_sync(1 + lt, 64);                       // the two warps of this quadrant
#pragma unroll
                for (int u = 0; u < KT; ++u) {
                    if (u != u_rt) continue;
#pragma unroll
                    for (int vi = 0; vi < VH; ++vi) {
                        const int vv = vi + half * VH;
                        if (vv >= KH) continue;
#pragma unroll
                        for (int ww = 0; ww < KW; ++ww)
                            sc[u][vi][ww] = stage[((ly + vv) * RX + lx + ww) * kPlQ + r] * lscale;
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            ok = __syncthreads_and(ok);                               // staging area and score buffer are free again
            if (!ok) break;
        }
        if (!ok) break;

        // ------------------------------------------------------------ softmax over the window (two threads per query)
        float mx = -INFINITY;
#pragma unroll
        for (int u = 0; u < KT; ++u)
#pragma unroll
            for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                for (int ww = 0; ww < KW; ++ww) mx = fmaxf(mx, sc[u][vi][ww]);
        s.pair_max[tid] = mx;
        named_barrier_sync(1 + lt, 64);
        mx = fmaxf(mx, s.pair_max[tid ^ 128]);
        float sum = 0.0f;
#pragma unroll
        for (int u = 0; u < KT; ++u)
#pragma unroll
            for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                for (int ww = 0; ww < KW; ++ww) {
                    sc[u][vi][ww] = exp2f(sc[u][vi][ww] - mx);            // cells this thread does not own: exp2(-inf) = 0
                    sum += sc[u][vi][ww];
                }
        s.pair_sum[tid] = sum;
        named_barrier_sync(1 + lt, 64);
        sum += s.pair_sum[tid ^ 128];
        const float inv = 1.0f / sum;
        const int qt = t0 + lt, qy = y0 + ly, qx = x0 + lx;
        const bool in_grid = qt < T && qy < H && qx < W;
        const long long n = (static_cast<long long>(qt) * H + qy) * W + qx;
        if (half == 0 && in_grid) lse[n * heads + m] = (mx + log2f(sum)) * kLn2;

        // ------------------------------------------------------------ pass 2: O += P_plane . V_plane
        // A thread's cells sit at the same columns of P in each of its KT planes, so its row only has
        // to be cleared before the first plane (the buffer held scores) and after its last one.
        const uint32_t row_off = static_cast<uint32_t>(r) * 128u, rx = static_cast<uint32_t>(r & 7);
        for (int pl = 0; pl < RT; ++pl) {
            const long long g = g0 + RT + pl, pvc = it * RT + pl;
            if (pl > 0) {
                if (!mbar_wait(smem_u32(&s.bar_pv), static_cast<uint32_t>((pvc - 1) & 1))) {
                    if (lane == 0) atomicExch(timeout_flag, 15);
                    ok = false;
                }
                if (tid == 0 && ok) issue_load(g + 1);                // the plane before this one has been multiplied
            }
            const int u_rt = pl - lt;
            const bool mine = u_rt >= 0 && u_rt < KT;
            if (pl == 0 || (!mine && u_rt == KT)) {                   // clear the row (one thread of the pair per matrix)
                unsigned char* dst = (half ? p_rest : p_head) + row_off;
#pragma unroll
                for (int c = 0; c < PSP / 8; ++c)
                    *reinterpret_cast<uint4*>(dst + (c >> 3) * (kPlQ * 128) + (((c & 7) ^ rx) << 4)) = make_uint4(0u, 0u, 0u, 0u);
            }
            if (pl == 0) named_barrier_sync(1 + lt, 64);              // both matrices of the row are clear before cells land
            if (mine) {
#pragma unroll
                for (int u = 0; u < KT; ++u) {
                    if (u != u_rt) continue;
#pragma unroll
                    for (int vi = 0; vi < VH; ++vi) {
                        const int vv = vi + half * VH;
                        if (vv >= KH) continue;
#pragma unroll
                        for (int ww = 0; ww < KW; ++ww) {
                            const float p = sc[u][vi][ww] * inv;
                            const __nv_bfloat16 hd = __float2bfloat16_rn(p);
                            const __nv_bfloat16 rs = __float2bfloat16_rn(p - __bfloat162float(hd));
                            const uint32_t col = static_cast<uint32_t>((ly + vv) * RX + lx + ww);
                            const uint32_t off = (col >> 6) * (kPlQ * 128) + row_off + ((((col & 63) >> 3) ^ rx) << 4) + (col & 7) * 2;
                            *reinterpret_cast<__nv_bfloat16*>(p_head + off) = hd;
                            *reinterpret_cast<__nv_bfloat16*>(p_rest + off) = rs;
                        }
                    }
                }
            }
            fence_async_smem();                                       // the MMAs read P through the async proxy
            ok = __syncthreads_and(ok);
            if (!ok) break;
            if (tid == 0) {
                if (full_wait(g)) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    constexpr uint32_t idesc = idesc_common | (1u << 16) | (static_cast<uint32_t>(D >> 3) << 17);   // B = V, MN-major
                    const uint64_t db = smem_desc_mn(smem_u32(s.slot[g & 1][0]), static_cast<uint32_t>(sizeof(s.slot[0][0])));
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        const uint32_t pa = smem_u32(part ? p_rest : p_head);
#pragma unroll
                        for (int ks = 0; ks < PSP / 16; ++ks)
                            umma_bf16(tmem, smem_desc(pa + (ks >> 2) * (kPlQ * 128)) + 2 * (ks & 3), db + 128 * ks, idesc,
                                      (pl | part | ks) ? 1u : 0u);
                    }
                } else {
                    atomicExch(timeout_flag, 16);
                    ok = false;
                }
                umma_commit(smem_u32(&s.bar_pv));
            }
        }
        ok = __syncthreads_and(ok);                                   // thread 0 may have given up on the last plane
        if (!ok) break;
        if (!mbar_wait(smem_u32(&s.bar_pv), static_cast<uint32_t>((it * RT + RT - 1) & 1))) {
            if (lane == 0) atomicExch(timeout_flag, 17);
            ok = false;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        ok = __syncthreads_and(ok);
        if (!ok) break;
        if (tid == 0) issue_load(g0 + JOBS + 1);                      // second plane of the next tile

        // ------------------------------------------------------------ epilogue: the pair splits the channels
        if (ok) {
            constexpr int CH = D / 2;                                 // channels per thread of the pair
#pragma unroll
            for (int c0 = 0; c0 < CH; c0 += 32) {
                uint32_t regs[32];
                tmem_load_32(tmem + lane_base + half * CH + c0, regs);
                if (in_grid) {
                    uint4* dst = reinterpret_cast<uint4*>(out + (n * heads + m) * D + half * CH + c0);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t o[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(regs[8 * i + 2 * j]),
                                                                            __uint_as_float(regs[8 * i + 2 * j + 1]));
                            o[j] = *reinterpret_cast<const uint32_t*>(&h2);
                        }
                        dst[i] = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        ok = __syncthreads_and(ok);                                   // O and the work area are free for the next tile
    }
    if (!ok && tid == 0) {            // stopped early: give loads still in flight a bounded time to land
        mbar_wait_limit(smem_u32(&s.bar_full[0]), 0u, 1u << 16);
        mbar_wait_limit(smem_u32(&s.bar_full[1]), 0u, 1u << 16);
        mbar_wait_limit(smem_u32(&s.bar_full[0]), 1u, 1u << 16);
        mbar_wait_limit(smem_u32(&s.bar_full[1]), 1u, 1u << 16);
        mbar_wait_limit(smem_u32(&s.bar_q), 0u, 1u << 16);
        mbar_wait_limit(smem_u32(&s.bar_q), 1u, 1u << 16);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
}

bool make_plane_maps(const void* q, const void* k, const void* v, const Problem& pr, int kh, int kw, CUtensorMap* mq,
                     CUtensorMap* mk, CUtensorMap* mv) {
    const unsigned long long d = static_cast<unsigned long long>(pr.d), hd = static_cast<unsigned long long>(pr.heads);
    const unsigned long long dims[5] = {d, hd, static_cast<unsigned long long>(pr.W), static_cast<unsigned long long>(pr.H),
                                        static_cast<unsigned long long>(pr.T)};
    const unsigned long long strides[4] = {d * 2, hd * d * 2, static_cast<unsigned long long>(pr.W) * hd * d * 2,
                                           static_cast<unsigned long long>(pr.H) * pr.W * hd * d * 2};
    const unsigned box_q[5] = {64, 1, kPlTX, kPlTY, kPlTT};
    const unsigned box_p[5] = {64, 1, static_cast<unsigned>(kPlTX + kw - 1), static_cast<unsigned>(kPlTY + kh - 1), 1};
    return encode_tensor_map_bf16(mq, q, 5, dims, strides, box_q, true) &&
           encode_tensor_map_bf16(mk, k, 5, dims, strides, box_p, true) &&
           encode_tensor_map_bf16(mv, v, 5, dims, strides, box_p, true);
}

template <int D, int KT, int KH, int KW>
cudaError_t launch_planes(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, void* out, float* lse,
                          const Problem& pr, int* flag, cudaStream_t stream) {
    const int tiles_x = (pr.W + kPlTX - 1) / kPlTX, tiles_y = (pr.H + kPlTY - 1) / kPlTY,
              tiles_t = (pr.T + kPlTT - 1) / kPlTT;
    const size_t smem = sizeof(PlSmem<D, KT, KH, KW>) + 1024;
    auto kern = fixed_window_planes_kernel<D, KT, KH, KW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kPlThreads, smem, stream>>>(mq, mk, mv, static_cast<__nv_bfloat16*>(out), lse, pr.T, pr.H, pr.W, pr.heads,
                                             tiles_x, tiles_y, total, flag);
    return cudaGetLastError();
}

}  // namespace

bool try_fixed_window_forward_planes(const void* q, const void* k, const void* v, void* out, float* lse,
                                     const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (pr.d != 128 && pr.d != 64) return false;
    const bool w355 = pr.kt == 3 && pr.kh == 5 && pr.kw == 5, w377 = pr.kt == 3 && pr.kh == 7 && pr.kw == 7;
    if (!w355 && !w377) return false;
    const long long tiles = static_cast<long long>((pr.W + kPlTX - 1) / kPlTX) * ((pr.H + kPlTY - 1) / kPlTY) *
                            ((pr.T + kPlTT - 1) / kPlTT);
    if (tiles > 0x7fffffffLL) return false;
    int* flag = timeout_flag_device_address();
    CUtensorMap mq, mk, mv;
    if (!flag || !make_plane_maps(q, k, v, pr, pr.kh, pr.kw, &mq, &mk, &mv)) return false;
    if (pr.d == 128)
        *err = w355 ? launch_planes<128, 3, 5, 5>(mq, mk, mv, out, lse, pr, flag, stream)
                    : launch_planes<128, 3, 7, 7>(mq, mk, mv, out, lse, pr, flag, stream);
    else
        *err = w355 ? launch_planes<64, 3, 5, 5>(mq, mk, mv, out, lse, pr, flag, stream)
                    : launch_planes<64, 3, 7, 7>(mq, mk, mv, out, lse, pr, flag, stream);
    return true;
}

}  // namespace dsa3d
