// Fixed-window backward (all offsets zero) for the larger windows - (3,5,5) and the paper's own
// (3,7,7) - with the three weighted sums of rows on the tensor cores:
//     dQ_i = sum_p ck_{i,p} K_{i+b(p)},   dK_j = sum_p ck_{j-b(p),p} q_{j-b(p)},   dV_j = sum_p cv_{j-b(p),p} dO_{j-b(p)}
// (ck = scale dS, cv = alpha: the two coefficients per sample that fixed_window_backward_query_kernel
// leaves; the chain rule of the Formulation with every sample on a grid position).  For a tile of
// 4 x 4 x 8 outputs each sum is  C . X_region  with C the coefficients placed at their region
// positions (zero elsewhere) - the forward's P . V with other weights and other rows - and the region
// (840 rows for (3,7,7)) is walked one plane (along t) at a time, exactly as the forward's second pass:
//
//   per (tile, head) three sweeps (dQ over K, dK over q, dV over dO), per sweep kt+3 planes:
//     the plane's rows by TMA into a ring of buffers; every worker thread writes the coefficients of
//     its output row that fall into this plane into the row of C_plane in shared memory
//     (128-byte-swizzled K-major), each fp32 coefficient split into a bf16 head and a bf16 remainder
//     (relative error of the pair 2^-17), as two matrices; two chains of tcgen05.mma (the plane as an
//     MN-major operand) accumulate  O_sweep += C_plane . X_plane  in TMEM - one accumulator per sweep,
//     so a sweep's epilogue (TMEM -> bf16 -> global) never holds up the next sweep's products.
//   The coefficients a thread needs for a plane are requested one plane ahead, with unconditional
//   loads from a clamped position (a load under a condition is waited for where it is issued).
//
// Roles: warps 0-7 are the workers (two threads per output row, the window's kernel rows split
// between them), warp 8 holds the thread that issues every TMA load, warp 9 the thread that issues
// every MMA.  Nothing but mbarriers orders the roles.  Every wait is bounded; a wait that runs out
// raises the library's timeout flag, after which nobody waits any more: the CTA walks through the
// rest of its work, drains its loads and frees its TMEM.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kPgTT = 4, kPgTY = 4, kPgTX = 8, kPgRows = kPgTT * kPgTY * kPgTX;    // 128 outputs per tile
constexpr int kPgWorkers = 256, kPgThreads = kPgWorkers + 64;
constexpr int kPgMaxSlots = 4;

template <int D, int KT, int KH, int KW>
struct PgShape {
    static constexpr int NH = D / 64;                               // 64-channel halves of a row
    static constexpr int RT = kPgTT + KT - 1, RY = kPgTY + KH - 1, RX = kPgTX + KW - 1;
    static constexpr int PS = RY * RX;                              // rows of one region plane
    static constexpr int PSP = (PS + 15) / 16 * 16;                 // padded to the MMA granularity
    static constexpr int KB = (PSP + 63) / 64;                      // 64-column blocks of a C row
    static constexpr int VH = (KH + 1) / 2;                         // kernel rows of the first thread of a pair
    static constexpr int C_BYTES = KB * kPgRows * 128;              // one coefficient matrix (head or remainder)
    static constexpr int SLOT_HALF = PSP * 128;                     // one 64-channel half of a plane buffer
    static constexpr int SLOT_BYTES = NH * SLOT_HALF;
    static constexpr int P = KT * KH * KW;
    // origin of the region below the tile: a gather (dQ) reaches k/2 back, a scatter seen from its
    // target (dK, dV) reaches k - 1 - k/2 back
    static constexpr int FT = KT / 2, FY = KH / 2, FX = KW / 2;
    static constexpr int BT = KT - 1 - KT / 2, BY = KH - 1 - KH / 2, BX = KW - 1 - KW / 2;
    static constexpr int NS_RAW = (227 * 1024 - 2048 - 2 * C_BYTES) / SLOT_BYTES;
    static constexpr int NS = NS_RAW > kPgMaxSlots ? kPgMaxSlots : NS_RAW;
    static_assert(PSP <= 256 && 3 * D <= 512, "a plane is one MMA's K extent; three accumulators in TMEM");
    static_assert(SLOT_HALF % 1024 == 0, "plane buffers keep the 1024-byte alignment of the swizzle");
    static_assert(NS >= 2, "at least two plane buffers");
    static_assert(VH * KW <= 32, "one bit per coefficient of a plane");
};

template <int D, int KT, int KH, int KW>
struct __align__(1024) PgSmem {
    using S = PgShape<D, KT, KH, KW>;
    unsigned char c[2][S::C_BYTES];                                 // coefficient matrix: head, remainder
    unsigned char slot[S::NS][S::NH][S::SLOT_HALF];                 // ring of region planes
    uint64_t bar_full[kPgMaxSlots], bar_slot_free[kPgMaxSlots];
    uint64_t bar_c_full[2], bar_c_free[2], bar_o[3];
    uint32_t tmem_base;
    uint32_t abort;                                                 // a wait ran out somewhere: nobody waits any more
};

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kPgThreads, 1)
fixed_window_planes_grad_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                                const __grid_constant__ CUtensorMap map_do, const float2* __restrict__ coef,
                                __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                                int T, int H, int W, int heads, int tiles_x, int tiles_y, int total, int* timeout_flag) {
    using S = PgShape<D, KT, KH, KW>;
    constexpr int NH = S::NH, RT = S::RT, RX = S::RX, PS = S::PS, PSP = S::PSP, VH = S::VH, NS = S::NS, P = S::P;
    constexpr int JOBS = 3 * RT;                                      // plane loads per tile
    extern __shared__ unsigned char raw[];
    PgSmem<D, KT, KH, KW>& s =
        *reinterpret_cast<PgSmem<D, KT, KH, KW>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kPgMaxSlots; ++i) { mbar_init(smem_u32(&s.bar_full[i]), 1); mbar_init(smem_u32(&s.bar_slot_free[i]), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s.bar_c_full[i]), kPgWorkers / 32);   // lane 0 of every worker warp
            mbar_init(smem_u32(&s.bar_c_free[i]), 1);
        }
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&s.bar_o[i]), 1);
        s.abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // the coefficient matrices start as zeros (a thread only ever writes its own cells, and writes them
    // back to zero after its last plane); rows PS .. PSP-1 of the plane buffers are never written by a
    // load and are multiplied by zero columns of C: they must not hold anything non-finite
    for (int i = tid; i < 2 * S::C_BYTES / 16; i += kPgThreads) reinterpret_cast<uint4*>(&s.c[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    if constexpr (PSP > PS) {
        for (int i = tid; i < NS * NH * (PSP - PS) * 8; i += kPgThreads) {
            const int chunk = i & 7, row = PS + (i >> 3) % (PSP - PS), which = (i >> 3) / (PSP - PS);
            *reinterpret_cast<uint4*>(&s.slot[which / NH][which % NH][row * 128 + chunk * 16]) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    fence_async_smem();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;
    volatile uint32_t* abort_flag = &s.abort;

    auto wait = [&](uint64_t* bar, uint32_t parity, int code) -> bool {
        if (*abort_flag) return false;
        if (mbar_wait(smem_u32(bar), parity)) return true;
        atomicExch(timeout_flag, code);
        *abort_flag = 1u;
        return false;
    };

    const int tiles_per_head = total / heads;                        // 32-bit throughout: the host checks the counts fit
    auto locate = [&](int ti, int& m, int& t0, int& y0, int& x0) {   // tile ti of this CTA
        const int item = static_cast<int>(blockIdx.x) + ti * static_cast<int>(gridDim.x);
        m = item / tiles_per_head;
        int tile = item - m * tiles_per_head;
        x0 = (tile % tiles_x) * kPgTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kPgTY;
        t0 = (tile / tiles_y) * kPgTT;
    };
    const int my_tiles = static_cast<int>(blockIdx.x) < total
                             ? (total - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;

    if (warp == kPgWorkers / 32) {
        // ==================================================================== loading thread (lane 0)
        if (lane == 0) {
            const int jobs_total = my_tiles * JOBS;
            int ti = 0, j = 0, m = 0, t0 = 0, y0 = 0, x0 = 0;
            if (my_tiles > 0) locate(0, m, t0, y0, x0);
            for (int g = 0; g < jobs_total; ++g) {
                const int sl = g % NS;
                if (g >= NS && !wait(&s.bar_slot_free[sl], static_cast<uint32_t>((g / NS - 1) & 1), 51)) break;
                const int sweep = j / RT, plane = j - sweep * RT;
                const uint32_t bar = smem_u32(&s.bar_full[sl]);
                mbar_expect_tx(bar, static_cast<uint32_t>(NH) * PS * 128u);
                const CUtensorMap* map = sweep == 0 ? &map_k : sweep == 1 ? &map_q : &map_do;
                const int ot = sweep == 0 ? S::FT : S::BT, oy = sweep == 0 ? S::FY : S::BY, ox = sweep == 0 ? S::FX : S::BX;
                for (int h = 0; h < NH; ++h)
                    tma_load_5d(smem_u32(s.slot[sl][h]), map, bar, h * 64, m, x0 - ox, y0 - oy, t0 - ot + plane);
                if (++j == JOBS) {
                    j = 0;
                    if (++ti < my_tiles) locate(ti, m, t0, y0, x0);
                }
            }
        }
    } else if (warp == kPgWorkers / 32 + 1) {
        // ==================================================================== MMA thread (lane 0)
        if (lane == 0) {
            // A = C (K-major bf16), B = the plane's rows (MN-major bf16), D = fp32, M = 128, N = D
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(D >> 3) << 17) |
                                       (static_cast<uint32_t>(kPgRows >> 4) << 24);
            constexpr uint64_t slot_step = S::SLOT_BYTES >> 4;
            uint64_t desc_c[2][S::KB];
            for (int part = 0; part < 2; ++part)
                for (int b = 0; b < S::KB; ++b) desc_c[part][b] = smem_desc(smem_u32(&s.c[part][b * (kPgRows * 128)]));
            const uint64_t desc_slot = smem_desc_mn(smem_u32(s.slot[0][0]), static_cast<uint32_t>(S::SLOT_HALF));
            int sl = 0, pc = 0;                                       // plane buffer, plane counter of the CTA
            uint32_t full_parity = 0;
            for (int it = 0; it < my_tiles; ++it) {
                for (int sweep = 0; sweep < 3; ++sweep) {
                    const uint32_t acc = tmem + static_cast<uint32_t>(sweep * D);
                    for (int pl = 0; pl < RT; ++pl, ++pc) {
                        bool ready = wait(&s.bar_full[sl], full_parity, 52);
#pragma unroll
                        for (int part = 0; part < 2; ++part) {
                            if (ready) ready = wait(&s.bar_c_full[part], static_cast<uint32_t>(pc & 1), 53);
                            if (ready) {
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                                for (int ks = 0; ks < PSP / 16; ++ks)
                                    umma_bf16(acc, desc_c[part][ks >> 2] + 2 * (ks & 3), desc_slot + sl * slot_step + 128 * ks, idesc,
                                              (pl | part | ks) ? 1u : 0u);
                            }
                            umma_commit(smem_u32(&s.bar_c_free[part]));   // arrives at once if nothing was issued
                        }
                        umma_commit(smem_u32(&s.bar_slot_free[sl]));
                        if (pl == RT - 1) umma_commit(smem_u32(&s.bar_o[sweep]));
                        if (++sl == NS) { sl = 0; full_parity ^= 1u; }
                    }
                }
            }
        }
    } else {
        // ==================================================================== workers
        const int lt = warp & 3, half = warp >> 2;                    // output plane of the tile; which thread of the pair
        const int ly = lane >> 3, lx = lane & 7;
        const int r = lt * 32 + lane;                                 // output row of the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>(lt * 32) << 16;
        const uint32_t row_off = static_cast<uint32_t>(r) * 128u, rx = static_cast<uint32_t>(r & 7);
        // byte offset, inside a coefficient matrix, of this row's cell at kernel row vv, column ww
        auto c_offset = [&](int vv, int ww) {
            const uint32_t col = static_cast<uint32_t>((ly + vv) * RX + lx + ww);
            return (col >> 6) * (kPgRows * 128) + row_off + ((((col & 63) >> 3) ^ rx) << 4) + (col & 7) * 2;
        };
        const float* cf = reinterpret_cast<const float*>(coef);
        // Step q of this thread = (tile, sweep, kernel plane u) in the order they come: the coefficients of
        // the row's cells (this thread's kernel rows, every column) in that plane.
        const int steps = my_tiles * 3 * KT;
        auto fetch = [&](int q, float (&wv)[VH][KW], uint32_t& dead) {
            const int ti = q / (3 * KT), rem = q - ti * (3 * KT), sweep = rem / KT, u = rem - sweep * KT;
            int m, t0, y0, x0;
            locate(ti, m, t0, y0, x0);
            const int ot = t0 + lt, oy = y0 + ly, ox = x0 + lx;       // the output position
            dead = 0u;
            long long base;                                           // index of the cell (first kernel row of this thread, column 0)
            int step_v, step_w;                                       // index steps to the next kernel row / column
            int st, sy0, sx0;                                         // the query the cell's coefficient belongs to
            if (sweep == 0) {                                         // output = the query itself, cell (u, vv, ww)
                st = ot; sy0 = oy; sx0 = ox;
                base = (((static_cast<long long>(ot) * H + oy) * W + ox) * heads + m) * P + (u * KH + half * VH) * KW;
                step_v = KW; step_w = 1;
            } else {                                                  // output = a key; the query at region offset (u, vv, ww) of it
                st = ot - S::BT + u; sy0 = oy - S::BY + half * VH; sx0 = ox - S::BX;
                base = (((static_cast<long long>(st) * H + sy0) * W + sx0) * heads + m) * P +
                       ((KT - 1 - u) * KH + (KH - 1 - half * VH)) * KW + (KW - 1);
                step_v = W * heads * P - KW; step_w = heads * P - 1;
            }
            const bool t_ok = st >= 0 && st < T;
            const float* src = cf + (sweep == 2 ? 1 : 0);
#pragma unroll
            for (int vi = 0; vi < VH; ++vi) {
                if (vi + half * VH >= KH) continue;                   // warp-uniform: the second thread of a pair has one row less
                const int sy = sweep == 0 ? sy0 : sy0 + vi;
                const bool ty_ok = t_ok && sy >= 0 && sy < H;
#pragma unroll
                for (int ww = 0; ww < KW; ++ww) {
                    const int sx = sweep == 0 ? sx0 : sx0 + ww;
                    const bool exists = ty_ok && sx >= 0 && sx < W;
                    const long long at = exists ? base + vi * step_v + ww * step_w : 0;
                    wv[vi][ww] = __ldg(src + 2 * at);
                    if (!exists) dead |= 1u << (vi * KW + ww);
                }
            }
        };

        float wnext[VH][KW], wcur[VH][KW];
        uint32_t dnext = 0u, dcur = 0u;
#pragma unroll
        for (int vi = 0; vi < VH; ++vi)
#pragma unroll
            for (int ww = 0; ww < KW; ++ww) wnext[vi][ww] = wcur[vi][ww] = 0.0f;
        int q = 0;                                                    // the step whose coefficients wnext holds
        if (steps > 0) fetch(0, wnext, dnext);
        int pc = 0;
        for (int it = 0; it < my_tiles; ++it) {
            int m, t0, y0, x0;
            locate(it, m, t0, y0, x0);
            const int ot = t0 + lt, oy = y0 + ly, ox = x0 + lx;
            const bool in_grid = ot < T && oy < H && ox < W;
            const long long n = (static_cast<long long>(ot) * H + oy) * W + ox;
            for (int sweep = 0; sweep < 3; ++sweep) {
                for (int pl = 0; pl < RT; ++pl, ++pc) {
                    const int u_rt = pl - lt;                         // the kernel plane this region plane is to the warp's outputs
                    const bool mine = u_rt >= 0 && u_rt < KT;
                    // cells go back to zero on the plane after the last; the last output plane of the tile has no
                    // such plane and clears its cells on the first plane of the next sweep instead
                    const bool clear = u_rt == KT || (lt == kPgTT - 1 && pl == 0);
                    if (mine) {
#pragma unroll
                        for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                            for (int ww = 0; ww < KW; ++ww) wcur[vi][ww] = wnext[vi][ww];
                        dcur = dnext;
                        if (++q < steps) fetch(q, wnext, dnext);
                    }
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        if (pc > 0) wait(&s.bar_c_free[part], static_cast<uint32_t>((pc - 1) & 1), 54);   // the chain of the plane before
                        if (mine || clear) {
                            unsigned char* dst = s.c[part];
#pragma unroll
                            for (int vi = 0; vi < VH; ++vi) {
                                const int vv = vi + half * VH;
                                if (vv >= KH) continue;
#pragma unroll
                                for (int ww = 0; ww < KW; ++ww) {
                                    const float p = (mine && !((dcur >> (vi * KW + ww)) & 1u)) ? wcur[vi][ww] : 0.0f;
                                    __nv_bfloat16 val = __float2bfloat16_rn(p);
                                    if (part) val = __float2bfloat16_rn(p - __bfloat162float(val));
                                    *reinterpret_cast<__nv_bfloat16*>(dst + c_offset(vv, ww)) = val;
                                }
                            }
                        }
                        fence_async_smem();                           // the MMAs read C through the async proxy
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&s.bar_c_full[part]));
                    }
                }
                // ------------------------------------------------------ epilogue of this sweep: the pair splits the channels
                wait(&s.bar_o[sweep], static_cast<uint32_t>(it & 1), 55);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                {
                    constexpr int CH = D / 2;
                    __nv_bfloat16* out = sweep == 0 ? dq : sweep == 1 ? dk : dv;
#pragma unroll
                    for (int c0 = 0; c0 < CH; c0 += 32) {
                        uint32_t regs[32];
                        tmem_load_32(tmem + lane_base + static_cast<uint32_t>(sweep * D + half * CH + c0), regs);
                        if (in_grid && !*abort_flag) {
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
            }
        }
    }
    // Gave up: loads may still be in flight towards this CTA's shared memory; give them a bounded time.
    if (*abort_flag && tid == kPgWorkers) {
        for (int i = 0; i < NS; ++i) {
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 0u, 1u << 16);
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 1u, 1u << 16);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
}

template <int D, int KT, int KH, int KW>
cudaError_t launch_planes_grad(const void* q, const void* k, const void* dout, const float2* coef, void* dq, void* dk, void* dv,
                               const Problem& pr, int* flag, cudaStream_t stream, bool* unsupported) {
    using S = PgShape<D, KT, KH, KW>;
    const unsigned long long d = static_cast<unsigned long long>(pr.d), hd = static_cast<unsigned long long>(pr.heads);
    const unsigned long long dims[5] = {d, hd, static_cast<unsigned long long>(pr.W), static_cast<unsigned long long>(pr.H),
                                        static_cast<unsigned long long>(pr.T)};
    const unsigned long long strides[4] = {d * 2, hd * d * 2, static_cast<unsigned long long>(pr.W) * hd * d * 2,
                                           static_cast<unsigned long long>(pr.H) * pr.W * hd * d * 2};
    const unsigned box[5] = {64, 1, static_cast<unsigned>(S::RX), static_cast<unsigned>(S::RY), 1};
    CUtensorMap mk, mq, mdo;
    if (!encode_tensor_map_bf16(&mk, k, 5, dims, strides, box, true) || !encode_tensor_map_bf16(&mq, q, 5, dims, strides, box, true) ||
        !encode_tensor_map_bf16(&mdo, dout, 5, dims, strides, box, true)) {
        *unsupported = true;
        return cudaSuccess;
    }
    const int tiles_x = (pr.W + kPgTX - 1) / kPgTX, tiles_y = (pr.H + kPgTY - 1) / kPgTY, tiles_t = (pr.T + kPgTT - 1) / kPgTT;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    // the kernel counts planes and coefficient indices relative to a row in 32 bits
    if (total * 3 * S::RT >= (1LL << 31) || static_cast<long long>(pr.W) * pr.heads * pr.P * (S::VH + 1) >= (1LL << 30)) {
        *unsupported = true;
        return cudaSuccess;
    }
    const size_t smem = sizeof(PgSmem<D, KT, KH, KW>) + 1024;
    auto kern = fixed_window_planes_grad_kernel<D, KT, KH, KW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kPgThreads, smem, stream>>>(mk, mq, mdo, coef, static_cast<__nv_bfloat16*>(dq), static_cast<__nv_bfloat16*>(dk),
                                             static_cast<__nv_bfloat16*>(dv), pr.T, pr.H, pr.W, pr.heads, tiles_x, tiles_y,
                                             static_cast<int>(total), flag);
    return cudaGetLastError();
}

}  // namespace

bool fixed_window_planes_grad_covers(const Problem& pr, bool bf16) {
    if (!bf16 || (pr.d != 128 && pr.d != 64)) return false;
    return pr.kt == 3 && ((pr.kh == 5 && pr.kw == 5) || (pr.kh == 7 && pr.kw == 7));
}

bool try_fixed_window_planes_grad(const void* q, const void* k, const void* dout, const float2* coef, void* dq, void* dk, void* dv,
                                  const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (!fixed_window_planes_grad_covers(pr, true)) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    const bool w355 = pr.kh == 5;
    if (pr.d == 128)
        *err = w355 ? launch_planes_grad<128, 3, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_planes_grad<128, 3, 7, 7>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    else
        *err = w355 ? launch_planes_grad<64, 3, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_planes_grad<64, 3, 7, 7>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    return !unsupported;
}

}  // namespace dsa3d
