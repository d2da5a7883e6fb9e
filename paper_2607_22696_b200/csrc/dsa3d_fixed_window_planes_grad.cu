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
//     (128-byte-swizzled K-major), each fp32 coefficient as a bf16 head and a bf16 remainder (relative
//     error of the pair 2^-17; the query kernel leaves them split like that), as two matrices; two
//     chains of tcgen05.mma (the plane as an MN-major operand) accumulate  O_sweep += C_plane . X_plane
//     in TMEM - one accumulator per sweep, so a sweep's epilogue (TMEM -> bf16 -> global) never holds
//     up the next sweep's products.
//   The coefficients a thread needs for a plane are requested one plane ahead, with unconditional
//   loads from a clamped position (a load under a condition is waited for where it is issued).
//
// Roles: warps 0-15 are the workers (four threads per output row, the window's kernel rows split
// between them: what bounds the kernel is the length of a worker's instruction stream per plane),
// warp 16 holds the thread that issues every TMA load, warp 17 the thread that issues every MMA.  Nothing but mbarriers orders the roles.  Every wait is bounded; a wait that runs out
// raises the library's timeout flag, after which nobody waits any more: the CTA walks through the
// rest of its work, drains its loads and frees its TMEM.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kPgTT = 4, kPgTY = 4, kPgTX = 8, kPgRows = kPgTT * kPgTY * kPgTX;    // 128 outputs per tile
constexpr int kPgSplit = 4;                                       // worker threads per output row (the window's kernel rows split between them)
constexpr int kPgWorkers = kPgSplit * kPgRows, kPgThreads = kPgWorkers + 64;
constexpr int kPgMaxSlots = 4;

template <int D, int KT, int KH, int KW>
struct PgShape {
    static constexpr int NH = D / 64;                               // 64-channel halves of a row
    static constexpr int RT = kPgTT + KT - 1, RY = kPgTY + KH - 1, RX = kPgTX + KW - 1;
    static constexpr int PS = RY * RX;                              // rows of one region plane
    static constexpr int PSP = (PS + 15) / 16 * 16;                 // padded to the MMA granularity
    static constexpr int KB = (PSP + 63) / 64;                      // 64-column blocks of a C row
    static constexpr int VH = (KH + kPgSplit - 1) / kPgSplit;       // kernel rows per worker thread, at most
    static constexpr int C_BYTES = KB * kPgRows * 128;              // one coefficient matrix (head or remainder)
    static constexpr int SLOT_HALF = PSP * 128;                     // one 64-channel half of a plane buffer
    static constexpr int SLOT_BYTES = NH * SLOT_HALF;
    static constexpr int P = KT * KH * KW;
    // origin of the region below the tile: a gather (dQ) reaches k/2 back, a scatter seen from its
    // target (dK, dV) reaches k - 1 - k/2 back
    static constexpr int FT = KT / 2, FY = KH / 2, FX = KW / 2;
    static constexpr int BT = KT - 1 - KT / 2, BY = KH - 1 - KH / 2, BX = KW - 1 - KW / 2;
    // The coefficient matrices of successive (plane, head | remainder) units rotate through NC buffers: the
    // workers write unit k + NC - 1 while the chain of unit k runs.  Two (head in one, remainder in the other)
    // measured best: every further buffer is one more unit in which a thread has to write its cells back to
    // zero after its last plane (3x5x5 backward 12.4 / 12.8 / 13.0 ms with 2 / 3 / 4), and leaves less room
    // for plane buffers.
    static constexpr int BUDGET = 227 * 1024 - 2048;
    static constexpr int NC = 2;
    static constexpr int NS_RAW = (BUDGET - NC * C_BYTES) / SLOT_BYTES;
    static constexpr int NS = NS_RAW > kPgMaxSlots ? kPgMaxSlots : NS_RAW;
    static_assert(PSP <= 256 && 3 * D <= 512, "a plane is one MMA's K extent; three accumulators in TMEM");
    static_assert(SLOT_HALF % 1024 == 0, "plane buffers keep the 1024-byte alignment of the swizzle");
    static_assert(NS >= 2, "at least two plane buffers");
    static_assert(VH * KW <= 32, "one bit per coefficient of a plane");
};

template <int D, int KT, int KH, int KW>
struct __align__(1024) PgSmem {
    using S = PgShape<D, KT, KH, KW>;
    unsigned char c[S::NC][S::C_BYTES];                             // coefficient matrices in rotation
    unsigned char slot[S::NS][S::NH][S::SLOT_HALF];                 // ring of region planes
    uint64_t bar_full[kPgMaxSlots], bar_slot_free[kPgMaxSlots];
    uint64_t bar_c_full[4], bar_c_free[4], bar_o[3];
    uint32_t tmem_base;
    uint32_t abort;                                                 // a wait ran out somewhere: nobody waits any more
};

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kPgThreads, 1)
fixed_window_planes_grad_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                                const __grid_constant__ CUtensorMap map_do, const uint32_t* __restrict__ coef,
                                __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                                int T, int H, int W, int heads, int tiles_x, int tiles_y, int total, int* timeout_flag,
                                const int* __restrict__ gate) {
    using S = PgShape<D, KT, KH, KW>;
    constexpr int NH = S::NH, RT = S::RT, RX = S::RX, PS = S::PS, PSP = S::PSP, VH = S::VH, NS = S::NS, NC = S::NC, P = S::P;
    constexpr int JOBS = 3 * RT;                                      // plane loads per tile
    extern __shared__ unsigned char raw[];
    PgSmem<D, KT, KH, KW>& s =
        *reinterpret_cast<PgSmem<D, KT, KH, KW>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kPgMaxSlots; ++i) { mbar_init(smem_u32(&s.bar_full[i]), 1); mbar_init(smem_u32(&s.bar_slot_free[i]), 1); }
        for (int i = 0; i < 4; ++i) {
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
    for (int i = tid; i < S::NC * S::C_BYTES / 16; i += kPgThreads) reinterpret_cast<uint4*>(&s.c[0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
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
    // behind a check of learned offsets: nothing to do unless the check left 0 in *gate
    const bool open = gate == nullptr || *gate == 0;
    const int my_tiles = open && static_cast<int>(blockIdx.x) < total
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
            uint64_t desc_c[NC][S::KB];
            for (int buf = 0; buf < NC; ++buf)
                for (int b = 0; b < S::KB; ++b) desc_c[buf][b] = smem_desc(smem_u32(&s.c[buf][b * (kPgRows * 128)]));
            const uint64_t desc_slot = smem_desc_mn(smem_u32(s.slot[0][0]), static_cast<uint32_t>(S::SLOT_HALF));
            int sl = 0, buf = 0;                                      // plane buffer; coefficient buffer of the next unit
            uint32_t full_parity = 0, c_parity = 0;
            for (int it = 0; it < my_tiles; ++it) {
                for (int sweep = 0; sweep < 3; ++sweep) {
                    const uint32_t acc = tmem + static_cast<uint32_t>(sweep * D);
                    for (int pl = 0; pl < RT; ++pl) {
                        bool ready = wait(&s.bar_full[sl], full_parity, 52);
#pragma unroll
                        for (int part = 0; part < 2; ++part) {
                            if (ready) ready = wait(&s.bar_c_full[buf], c_parity, 53);
                            if (ready) {
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                // one of NC descriptor sets; chosen by comparisons so that the array stays in registers
                                uint64_t dc[S::KB];
#pragma unroll
                                for (int b = 0; b < S::KB; ++b) {
                                    dc[b] = desc_c[0][b];
#pragma unroll
                                    for (int i = 1; i < NC; ++i) if (buf == i) dc[b] = desc_c[i][b];
                                }
#pragma unroll
                                for (int ks = 0; ks < PSP / 16; ++ks)
                                    umma_bf16(acc, dc[ks >> 2] + 2 * (ks & 3), desc_slot + sl * slot_step + 128 * ks, idesc,
                                              (pl | part | ks) ? 1u : 0u);
                            }
                            umma_commit(smem_u32(&s.bar_c_free[buf]));    // arrives at once if nothing was issued
                            if (++buf == NC) { buf = 0; c_parity ^= 1u; }
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
        // A worker thread has two places.  Writing coefficients it is thread `sub` of the four that share the
        // output row (lt, lane); the four warps of one lt sit on four different schedulers, so the planes a
        // row group is busy in load all of them.  Reading an accumulator it can only reach the TMEM lanes of
        // its warp's quarter (warp % 4): there it takes 32 channels (part warp / 4) of row (warp % 4, lane).
        const int lt = warp >> 2, sub = warp & 3;                     // output plane of the tile; which thread of the row's four
        const int lt_acc = warp & 3, part_acc = warp >> 2;
        const int ly = lane >> 3, lx = lane & 7;
        const int r = lt * 32 + lane;                                 // output row of the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>(lt_acc * 32) << 16;
        const uint32_t row_off = static_cast<uint32_t>(r) * 128u, rx = static_cast<uint32_t>(r & 7);
        const int v0 = (sub * KH) / kPgSplit, nv = ((sub + 1) * KH) / kPgSplit - v0;    // this thread's kernel rows (warp-uniform)
        // The cells of one kernel row are KW neighbouring columns of the output's row of C: they are written as
        // whole 16-byte chunks of 8 columns (one chunk, or two when the cells straddle a chunk boundary).
        // The other columns of those chunks belong to no cell of this output row - the neighbouring kernel
        // rows lie 8 + KW - 1 columns away - so writing them as zeros is right.  Where the chunks lie and by
        // how many columns the cells are shifted inside them is the same for every plane and tile:
        // bits 0-11 / 12-23 the byte offsets of the two chunks (in 16-byte units), bits 24-26 the shift.
        static_assert(S::C_BYTES <= 65536 && KW <= 7 && RX >= KW + 7, "chunk offsets in 12 bits; a kernel row's chunks touch no other row's cells");
        constexpr int CELLS = VH * KW;
        uint32_t row_geo[VH];
#pragma unroll
        for (int vi = 0; vi < VH; ++vi) {
            const int vv = vi < nv ? v0 + vi : v0;
            const uint32_t col0 = static_cast<uint32_t>((ly + vv) * RX + lx);
            auto chunk_off = [&](uint32_t col) { return (col >> 6) * (kPgRows * 128) + row_off + ((((col & 63) >> 3) ^ rx) << 4); };
            row_geo[vi] = (chunk_off(col0) >> 4) | ((chunk_off(col0 + 8) >> 4) << 12) | ((col0 & 7u) << 24);
        }
        // The KW cells of a kernel row (a word each: bf16 head | bf16 remainder << 16) moved to their places among
        // the 16 columns of the row's two chunks - one network of selects for head and remainder together, the
        // shift (0 .. 7 columns) being the thread's own - then parted into the words of the head matrix and of
        // the remainder matrix (two columns per word).
        auto align_row = [&](uint32_t geo, const uint32_t (&cell)[8], uint32_t (&head)[8], uint32_t (&rest)[8]) {
            const bool s1 = (geo >> 24) & 1u, s2 = (geo >> 25) & 1u, s4 = (geo >> 26) & 1u;
            uint32_t a[8], b[10], c[14];
            a[0] = s1 ? 0u : cell[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) a[i] = s1 ? cell[i - 1] : cell[i];              // cell[7] is always 0 (KW <= 7)
#pragma unroll
            for (int i = 0; i < 10; ++i) b[i] = s2 ? (i >= 2 ? a[i - 2] : 0u) : (i < 8 ? a[i] : 0u);
#pragma unroll
            for (int i = 0; i < 14; ++i) c[i] = s4 ? (i >= 4 ? b[i - 4] : 0u) : (i < 10 ? b[i] : 0u);
#pragma unroll
            for (int j = 0; j < 7; ++j) {
                head[j] = __byte_perm(c[2 * j], c[2 * j + 1], 0x5410);
                rest[j] = __byte_perm(c[2 * j], c[2 * j + 1], 0x7632);
            }
            head[7] = rest[7] = 0u;
        };
        auto store_chunks = [&](unsigned char* dst, uint32_t geo, const uint32_t (&w)[8]) {
            *reinterpret_cast<uint4*>(dst + ((geo & 0xfffu) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            if (((geo >> 24) & 7u) + KW > 8u) *reinterpret_cast<uint4*>(dst + (((geo >> 12) & 0xfffu) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        };
        const int n_step = T * H * W;                                 // tokens: the step from one sample's plane to the next
        const uint32_t* plane_ck = coef;                              // [head][sample][token], a word = bf16 head | bf16 remainder << 16
        const uint32_t* plane_cv = coef + static_cast<long long>(heads) * P * n_step;
        // Step q of this thread = (tile, sweep, kernel plane u) in the order they come: the coefficients of
        // the row's cells (this thread's kernel rows, every column) in that plane.  What depends on the
        // tile alone is worked out at the tile's first step: positions inside a coefficient plane (they
        // fit 32 bits, the host checks) and which source queries exist.
        const int steps = my_tiles * 3 * KT;
        int g_a0 = 0, g_a1 = 0;
        uint32_t g_tmask = 0u, g_ymask = 0u, g_xmask = 0u, g_own = 0u;
        auto fetch = [&](int q, uint32_t (&wv)[CELLS], uint32_t& dead) {
            const int ti = q / (3 * KT), rem = q - ti * (3 * KT), sweep = rem / KT, u = rem - sweep * KT;
            if (rem == 0) {
                int m, t0, y0, x0;
                locate(ti, m, t0, y0, x0);
                const int ot = t0 + lt, oy = y0 + ly, ox = x0 + lx;   // the output position
                const int n_out = (ot * H + oy) * W + ox;
                g_a0 = m * P * n_step + n_out;                        // sample 0 of the output's own query
                g_a1 = (m * P + P - 1) * n_step + n_out - ((S::BT * H + S::BY) * W + S::BX);   // last sample of the first source query
                g_own = (ot < T && oy < H && ox < W) ? (1u << KW) - 1u : 0u;
                g_tmask = g_ymask = g_xmask = 0u;
#pragma unroll
                for (int i = 0; i < KT; ++i) if (ot - S::BT + i >= 0 && ot - S::BT + i < T) g_tmask |= 1u << i;
#pragma unroll
                for (int i = 0; i < VH; ++i) if (i < nv && oy - S::BY + v0 + i >= 0 && oy - S::BY + v0 + i < H) g_ymask |= 1u << i;
#pragma unroll
                for (int i = 0; i < KW; ++i) if (ox - S::BX + i >= 0 && ox - S::BX + i < W) g_xmask |= 1u << i;
            }
            // sweep 0: the output is the query itself, cell (u, v0 + vi, ww) = sample index, own token;
            // sweeps 1, 2: the output is a key, the cell at region offset (u, v0 + vi, ww) belongs to the query
            // at that offset from (key - B) and is its sample mirrored in the window
            int base, step_v, step_w;
            uint32_t alive = 0u;
            if (sweep == 0) {
                base = g_a0 + (u * KH + v0) * KW * n_step;
                step_v = KW * n_step; step_w = n_step;
#pragma unroll
                for (int vi = 0; vi < VH; ++vi) if (vi < nv) alive |= g_own << (vi * KW);
            } else {
                base = g_a1 + u * (H * W - KH * KW * n_step) + v0 * (W - KW * n_step);
                step_v = W - KW * n_step; step_w = 1 - n_step;
                if ((g_tmask >> u) & 1u) {
#pragma unroll
                    for (int vi = 0; vi < VH; ++vi) if ((g_ymask >> vi) & 1u) alive |= g_xmask << (vi * KW);
                }
            }
            const uint32_t* plane = sweep == 2 ? plane_cv : plane_ck;
#pragma unroll
            for (int i = 0; i < CELLS; ++i) {
                const int vi = i / KW, ww = i - vi * KW;
                const int at = ((alive >> i) & 1u) ? base + vi * step_v + ww * step_w : 0;    // a cell that does not exist reads word 0
                wv[i] = __ldg(plane + at);
            }
            dead = ~alive;
        };
        uint32_t wnext[CELLS];
        uint32_t dnext = 0u;
#pragma unroll
        for (int i = 0; i < CELLS; ++i) wnext[i] = 0u;
        int q = 0;                                                    // the step whose coefficients wnext holds
        if (steps > 0) fetch(0, wnext, dnext);
        int buf = 0, clear_left = 0;                                  // coefficient buffer of the next unit; units still to clear
        uint32_t c_parity = 0;
        bool first_round = true;                                      // the first NC units find their buffers free
        // Epilogue of sweep `sweep` of this CTA's tile `it`: the row's threads split the channels.
        auto epilogue = [&](int it, int sweep) {
            int m, t0, y0, x0;
            locate(it, m, t0, y0, x0);
            const int ot = t0 + lt_acc, oy = y0 + ly, ox = x0 + lx;
            const bool in_grid = ot < T && oy < H && ox < W;
            const long long n = (static_cast<long long>(ot) * H + oy) * W + ox;
            wait(&s.bar_o[sweep], static_cast<uint32_t>(it & 1), 55);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (part_acc * 32 < D) {
                __nv_bfloat16* out = sweep == 0 ? dq : sweep == 1 ? dk : dv;
                uint32_t regs[32];
                tmem_load_32(tmem + lane_base + static_cast<uint32_t>(sweep * D + part_acc * 32), regs);
                if (in_grid && !*abort_flag) {
                    uint4* dst = reinterpret_cast<uint4*>(out + (n * heads + m) * D + part_acc * 32);
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
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        };
        // The planes of the CTA's tiles and sweeps form one stream.  The epilogue of a sweep is taken after
        // the first plane of the next sweep has been written, so that the MMA thread has that plane's chains
        // to run meanwhile (each sweep has its own accumulator; by then the sweep's last chain is usually done).
        for (int pj = 0, it = 0, sweep = 0, pl = 0; it < my_tiles; ++pj) {
            const int u_rt = pl - lt;                         // the kernel plane this region plane is to the warp's outputs
            const bool mine = u_rt >= 0 && u_rt < KT;
            // A thread's cells are the same columns in every unit.  After its last plane of a sweep it
            // writes them back to zero in the NC units that follow (one per buffer).
            const bool writes = mine || clear_left > 0;
            uint32_t rest[VH][8];                             // remainder words of this plane's rows, already in place
            // ---- head
            if (!first_round) wait(&s.bar_c_free[buf], c_parity ^ 1u, 54);       // the chain of the unit NC before this one
            if (writes) {
                unsigned char* dst = s.c[buf];
#pragma unroll
                for (int vi = 0; vi < VH; ++vi) {
                    if (vi >= nv) continue;
                    // the row's cells: 0 beyond KW, for a query that does not exist, and when clearing
                    uint32_t cell[8], head[8];
#pragma unroll
                    for (int ww = 0; ww < 8; ++ww) {
                        const int i = vi * KW + (ww < KW ? ww : 0);
                        cell[ww] = (ww < KW && mine && !((dnext >> i) & 1u)) ? wnext[i] : 0u;
                    }
                    align_row(row_geo[vi], cell, head, rest[vi]);
                    store_chunks(dst, row_geo[vi], head);
                }
                if (!mine) --clear_left;
            }
            fence_async_smem();                               // the MMAs read C through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_c_full[buf]));
            if (++buf == NC) { buf = 0; c_parity ^= 1u; first_round = false; }
            // the next plane's coefficients: requested once the head is out, on their way while the
            // remainder is written and through the waits of the next plane
            if (mine && ++q < steps) fetch(q, wnext, dnext);
            // ---- remainder
            const bool writes_rest = mine || clear_left > 0;
            if (!first_round) wait(&s.bar_c_free[buf], c_parity ^ 1u, 54);
            if (writes_rest) {
                unsigned char* dst = s.c[buf];
                const uint32_t zero[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                for (int vi = 0; vi < VH; ++vi) {
                    if (vi >= nv) continue;
                    if (mine) store_chunks(dst, row_geo[vi], rest[vi]);
                    else store_chunks(dst, row_geo[vi], zero);
                }
                if (!mine) --clear_left;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_c_full[buf]));
            if (++buf == NC) { buf = 0; c_parity ^= 1u; first_round = false; }
            if (mine && u_rt == KT - 1) clear_left = NC;
            if (pl == 0 && pj > 0) epilogue(sweep == 0 ? it - 1 : it, sweep == 0 ? 2 : sweep - 1);
            if (++pl == RT) {
                pl = 0;
                if (++sweep == 3) { sweep = 0; ++it; }
            }
        }
        if (my_tiles > 0) epilogue(my_tiles - 1, 2);
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
cudaError_t launch_planes_grad(const void* q, const void* k, const void* dout, const uint32_t* coef, void* dq, void* dk, void* dv,
                               const Problem& pr, int* flag, cudaStream_t stream, bool* unsupported, const int* gate = nullptr) {
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
    // the kernel counts planes, and positions inside a coefficient plane, in 32 bits
    if (total * 3 * S::RT >= (1LL << 31) || pr.N * pr.heads * S::P >= (1LL << 31)) {
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
                                             static_cast<int>(total), flag, gate);
    return cudaGetLastError();
}

}  // namespace

bool fixed_window_planes_grad_covers(const Problem& pr, bool bf16) {
    if (!bf16 || (pr.d != 128 && pr.d != 64)) return false;
    return pr.kt == 3 && ((pr.kh == 5 && pr.kw == 5) || (pr.kh == 7 && pr.kw == 7));
}

bool try_fixed_window_planes_grad(const void* q, const void* k, const void* dout, const float* coef_planes, void* dq, void* dk, void* dv,
                                  const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (!fixed_window_planes_grad_covers(pr, true)) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    const uint32_t* coef = reinterpret_cast<const uint32_t*>(coef_planes);
    const bool w355 = pr.kh == 5;
    if (pr.d == 128)
        *err = w355 ? launch_planes_grad<128, 3, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_planes_grad<128, 3, 7, 7>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    else
        *err = w355 ? launch_planes_grad<64, 3, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported)
                    : launch_planes_grad<64, 3, 7, 7>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported);
    return !unsupported;
}

// Learned offsets below 1 in size, window (3,3,3): the coefficients of a query's samples, summed per grid
// position, fill the box of 5 x 5 x 5 positions around the query; dQ, dK and dV are then the sums of a
// fixed (5,5,5) window with those coefficients.  `coef_planes`: ck and cv planes [head][125][token].
bool try_bounded_offsets_planes_grad(const void* q, const void* k, const void* dout, const float* coef_planes, void* dq,
                                     void* dk, void* dv, const Problem& pr, const int* gate, cudaStream_t stream,
                                     cudaError_t* err) {
    *err = cudaSuccess;
    if ((pr.d != 128 && pr.d != 64) || pr.kt != 3 || pr.kh != 3 || pr.kw != 3) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    const uint32_t* coef = reinterpret_cast<const uint32_t*>(coef_planes);
    *err = pr.d == 128 ? launch_planes_grad<128, 5, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported, gate)
                       : launch_planes_grad<64, 5, 5, 5>(q, k, dout, coef, dq, dk, dv, pr, flag, stream, &unsupported, gate);
    return !unsupported;
}

}  // namespace dsa3d
