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
//     the two warps that share a TMEM quadrant (= the 32 queries of one tile plane) copy the
//     plane's score columns to shared memory, every thread picks the window cells of its query
//     that lie in this plane (static register indices).  Two threads serve a query (the window's
//     kernel rows are split between them).
//   softmax in registers; the pair of threads exchanges max and sum through shared memory; lse out.
//   pass 2, plane by plane:  V plane by TMA into the same ring of buffers; every thread writes its
//     cells into its query's row of P_plane in shared memory (128-byte-swizzled K-major layout),
//     each fp32 weight split into a bf16 head and a bf16 remainder (relative error of the pair
//     2^-17, far inside the rounding of the output), as two matrices; two chains of tcgen05.mma
//     (V as an MN-major operand) accumulate  O += P_plane . V_plane  in TMEM.  While the chain of
//     one matrix runs, the other matrix is being written.
//   epilogue: O from TMEM, one rounding to bf16, out.
//
// Roles: warps 0-7 are the workers described above; warp 8 holds the one thread that issues every
// TMA load and every MMA.  Nothing but mbarriers (and a barrier per pair of worker warps) orders the
// roles inside a tile, so a quadrant only stops at the planes its own queries see.  Every wait on
// an mbarrier is bounded; a wait that runs out raises the library's timeout flag, the CTA walks
// through the rest of its tile without waiting, drains its loads and frees its TMEM.
#include <cuda_bf16.h>

#include <type_traits>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kPlTT = 4, kPlTY = 4, kPlTX = 8, kPlQ = kPlTT * kPlTY * kPlTX;    // 128 queries per tile
constexpr int kPlWorkers = 256, kPlThreads = kPlWorkers + 64;      // + loading warp + MMA warp
constexpr int kPlMaxSlots = 4;

// BOUNDED = false: fixed window (KT, KH, KW), all offsets zero.  BOUNDED = true: learned offsets with
// |offset| < 1 on every axis; (KT, KH, KW) is then the BOX of grid positions a query's samples can touch,
// the window grown by one position on each side, and the window itself is (KT-2, KH-2, KW-2).
template <int D, int KT, int KH, int KW, bool BOUNDED = false>
struct PlaneShape {
    static constexpr int NH = D / 64;                               // 64-channel halves of a row
    static constexpr int RT = kPlTT + KT - 1, RY = kPlTY + KH - 1, RX = kPlTX + KW - 1;
    static constexpr int PS = RY * RX;                              // key rows of one region plane
    static constexpr int PSP = (PS + 15) / 16 * 16;                 // padded to the MMA granularity
    static constexpr int KB = (PSP + 63) / 64;                      // 64-column blocks of a P row
    static constexpr int PIECES = (PS + 31) / 32;                   // 32-column pieces of a score plane
    static constexpr int VH = (KH + 1) / 2;                         // kernel rows of the first thread of a pair
    static constexpr int SBUF = PIECES * 32;                        // TMEM columns set aside per score buffer
    static constexpr int S0 = D, S1 = D + SBUF;                     // TMEM: O at 0, two score buffers behind it
    static constexpr int P_BYTES = KB * kPlQ * 128;                 // one P matrix (head or remainder)
    static constexpr int STAGE_BYTES = PIECES * 32 * kPlQ * 4;      // a score plane as [column][query] floats
    static constexpr int Q_BYTES = NH * kPlQ * 128;
    static constexpr int SLOT_HALF = PSP * 128;                     // one 64-channel half of a plane buffer
    static constexpr int SLOT_BYTES = NH * SLOT_HALF;
    static constexpr int CELLS = KT * KH * KW;
    static constexpr int BOX_BYTES = BOUNDED ? CELLS * kPlQ * 4 : 0;       // per query: scores, then weights, of its box
    static constexpr int SMALL_BYTES = 2 * kPlWorkers * 4 + 256 + 2048 + BOX_BYTES;   // pair arrays, barriers, slack, box
    static constexpr int BUDGET = 227 * 1024;
    // Work area: the score staging of pass 1 and the two P matrices of pass 2 share their bytes.
    // Q has its own buffer (so the next tile's Q arrives during pass 2) unless giving it up buys
    // a third plane buffer: then it sits behind the staging area, on top of the tail of P.
    static constexpr int WORK_OWN = (2 * P_BYTES > STAGE_BYTES ? 2 * P_BYTES : STAGE_BYTES);
    static constexpr int NS_OWN = (BUDGET - SMALL_BYTES - Q_BYTES - WORK_OWN) / SLOT_BYTES;
    static constexpr int WORK_SHARED = (2 * P_BYTES > STAGE_BYTES + Q_BYTES ? 2 * P_BYTES : STAGE_BYTES + Q_BYTES);
    static constexpr int NS_SHARED = (BUDGET - SMALL_BYTES - WORK_SHARED) / SLOT_BYTES;
    static constexpr bool Q_SHARED = NS_OWN < 3 && NS_SHARED > NS_OWN;
    static constexpr int NS_RAW = Q_SHARED ? NS_SHARED : NS_OWN;
    static constexpr int NS = NS_RAW > kPlMaxSlots ? kPlMaxSlots : NS_RAW;
    static constexpr int WORK_BYTES = Q_SHARED ? WORK_SHARED : WORK_OWN;
    static constexpr int Q_OFFSET = STAGE_BYTES;                    // of Q inside the work area when shared
    static_assert(PSP <= 256, "a region plane must fit one MMA (N <= 256)");
    static_assert(D + 2 * SBUF <= 512, "TMEM columns");
    static_assert(SLOT_HALF % 1024 == 0 && STAGE_BYTES % 1024 == 0, "buffers keep the 1024-byte alignment of the swizzle");
    static_assert(NS >= 2, "at least two plane buffers");
};

template <int D, int KT, int KH, int KW, bool BOUNDED = false>
struct __align__(1024) PlSmem {
    using S = PlaneShape<D, KT, KH, KW, BOUNDED>;
    unsigned char work[S::WORK_BYTES];                              // staging (pass 1) / P head + remainder (pass 2) [/ Q]
    unsigned char slot[S::NS][S::NH][S::SLOT_HALF];                 // ring of K or V planes, same image for both uses
    unsigned char q_own[S::Q_SHARED ? 1024 : S::Q_BYTES];           // 64-channel halves, swizzled 128-byte rows
    float box[BOUNDED ? S::CELLS * kPlQ : 1];                      // [cell][query]
    float pair_max[kPlWorkers], pair_sum[kPlWorkers];
    uint64_t bar_q, bar_full[kPlMaxSlots], bar_slot_free[kPlMaxSlots];
    uint64_t bar_s[2], bar_s_free[2], bar_p_full[2], bar_p_free[2], bar_o;
    uint32_t tmem_base;
    uint32_t abort;                                                 // a wait ran out somewhere: nobody waits any more
};

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Barrier 6 of the workers and the MMA warp at the end of a tile; returns the OR of `flag` over them.
__device__ __forceinline__ bool tile_barrier_or(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 6, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"(static_cast<uint32_t>(flag)), "r"(kPlWorkers + 32) : "memory");
    return out != 0u;
}

template <int D, int KT, int KH, int KW, bool BOUNDED>
__global__ void __launch_bounds__(kPlThreads, 1)
fixed_window_planes_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ out,
                           float* __restrict__ lse, int T, int H, int W, int heads, int tiles_x, int tiles_y,
                           int total, int* timeout_flag, const float* __restrict__ offsets, const int* __restrict__ gate) {
    using S = PlaneShape<D, KT, KH, KW, BOUNDED>;
    constexpr int NH = S::NH, RT = S::RT, RX = S::RX, PS = S::PS, PSP = S::PSP, VH = S::VH, NS = S::NS;
    constexpr int JOBS = 2 * RT;                                      // plane loads per tile: RT of K, then RT of V
    extern __shared__ unsigned char raw[];
    PlSmem<D, KT, KH, KW, BOUNDED>& s =
        *reinterpret_cast<PlSmem<D, KT, KH, KW, BOUNDED>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* q_buf = S::Q_SHARED ? s.work + S::Q_OFFSET : s.q_own;
    unsigned char* p_head = s.work;
    unsigned char* p_rest = s.work + S::P_BYTES;

    if (tid == 0) {
        mbar_init(smem_u32(&s.bar_q), 1);
        for (int i = 0; i < kPlMaxSlots; ++i) { mbar_init(smem_u32(&s.bar_full[i]), 1); mbar_init(smem_u32(&s.bar_slot_free[i]), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s.bar_s[i]), 1);
            mbar_init(smem_u32(&s.bar_s_free[i]), kPlWorkers / 32);   // lane 0 of every worker warp
            mbar_init(smem_u32(&s.bar_p_full[i]), kPlWorkers / 32);   // lane 0 of every worker warp
            mbar_init(smem_u32(&s.bar_p_free[i]), 1);
        }
        mbar_init(smem_u32(&s.bar_o), 1);
        s.abort = 0u;
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
        for (int i = tid; i < NS * NH * (PSP - PS) * 8; i += kPlThreads) {
            const int chunk = i & 7, row = PS + (i >> 3) % (PSP - PS), which = (i >> 3) / (PSP - PS);
            *reinterpret_cast<uint4*>(&s.slot[which / NH][which % NH][row * 128 + chunk * 16]) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;
    volatile uint32_t* abort_flag = &s.abort;

    // A wait of this kernel: skipped once somebody has given up (the tile is then walked through
    // without waiting and thrown away); a wait that runs out raises the flags itself.
    auto wait = [&](uint64_t* bar, uint32_t parity, int code) -> bool {
        if (*abort_flag) return false;
        if (mbar_wait(smem_u32(bar), parity)) return true;
        atomicExch(timeout_flag, code);
        *abort_flag = 1u;
        return false;
    };

    const int tiles_per_head = total / heads;                        // 32-bit throughout: the host checks the counts fit
    auto locate = [&](int item, int& m, int& t0, int& y0, int& x0) {
        m = item / tiles_per_head;
        int tile = item - m * tiles_per_head;
        x0 = (tile % tiles_x) * kPlTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kPlTY;
        t0 = (tile / tiles_y) * kPlTT;
    };
    // BOUNDED: an earlier kernel on the stream left 0 in *gate if every offset is finite and below 1 in size;
    // otherwise this kernel has nothing to do (the general kernel runs instead)
    const bool open = !BOUNDED || gate == nullptr || *gate == 0;
    const int my_tiles = (open && static_cast<int>(blockIdx.x) < total)
                             ? (total - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;

    if (warp == kPlWorkers / 32) {
        // ==================================================================== loading thread (lane 0)
        // Walks the CTA's stream of plane loads (tile after tile: RT planes of K, RT planes of V) as
        // far ahead as the ring of plane buffers allows, and puts the Q loads in between.  It takes no
        // part in the per-tile barrier of the other roles.
        if (lane == 0 && my_tiles > 0) {
            const int jobs_total = my_tiles * JOBS;
            int tile_index = 0, j = 0;                               // tile and plane load within it of load g
            int m, t0, y0, x0;
            auto locate_tile = [&](int ti) { locate(static_cast<int>(blockIdx.x) + ti * static_cast<int>(gridDim.x), m, t0, y0, x0); };
            auto load_q = [&](int ti) {
                int qm, qt0, qy0, qx0;
                locate(static_cast<int>(blockIdx.x) + ti * static_cast<int>(gridDim.x), qm, qt0, qy0, qx0);
                mbar_expect_tx(smem_u32(&s.bar_q), static_cast<uint32_t>(NH) * kPlQ * 128u);
                for (int h = 0; h < NH; ++h)
                    tma_load_5d(smem_u32(q_buf + h * (kPlQ * 128)), &map_q, smem_u32(&s.bar_q), h * 64, qm, qx0, qy0, qt0);
            };
            // Q of tile ti + 1 may be loaded once the MMAs of plane load `q_free_job` of tile ti have run:
            // the tile's last score plane, or - when Q lies on the tail of P - its last P.V plane.
            constexpr int q_free_job = S::Q_SHARED ? JOBS - 1 : RT - 1;
            locate_tile(0);
            load_q(0);
            for (int g = 0; g < jobs_total; ++g) {
                const int sl = g % NS;
                if (g >= NS) {
                    if (!wait(&s.bar_slot_free[sl], static_cast<uint32_t>((g / NS - 1) & 1), 13)) break;
                    // the MMAs of load g - NS have run
                    const int done = g - NS, done_tile = done / JOBS;
                    if (done - done_tile * JOBS == q_free_job && done_tile + 1 < my_tiles) load_q(done_tile + 1);
                }
                const uint32_t bar = smem_u32(&s.bar_full[sl]);
                mbar_expect_tx(bar, static_cast<uint32_t>(NH) * PS * 128u);
                const CUtensorMap* map = j < RT ? &map_k : &map_v;
                const int plane = j < RT ? j : j - RT;
                for (int h = 0; h < NH; ++h)
                    tma_load_5d(smem_u32(s.slot[sl][h]), map, bar, h * 64, m, x0 - KW / 2, y0 - KH / 2, t0 - KT / 2 + plane);
                if (++j == JOBS) {
                    j = 0;
                    if (++tile_index < my_tiles) locate_tile(tile_index);
                }
            }
            // Q loads whose trigger lies within the last NS plane loads of the stream
            if (!*abort_flag) {
                for (int done = jobs_total - NS < 0 ? 0 : jobs_total - NS; done < jobs_total; ++done) {
                    const int done_tile = done / JOBS;
                    if (done - done_tile * JOBS == q_free_job && done_tile + 1 < my_tiles) {
                        if (wait(&s.bar_slot_free[done % NS], static_cast<uint32_t>((done / NS) & 1), 13)) load_q(done_tile + 1);
                    }
                }
            }
        }
    } else if (warp == kPlWorkers / 32 + 1) {
        // ==================================================================== MMA thread (lane 0)
        constexpr uint32_t idesc_common = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kPlQ >> 4) << 24);
        constexpr uint32_t idesc_s = idesc_common | (static_cast<uint32_t>(PSP >> 3) << 17);
        constexpr uint32_t idesc_pv = idesc_common | (1u << 16) | (static_cast<uint32_t>(D >> 3) << 17);     // B = V, MN-major
        // descriptors of plane buffer 0; buffer i lies i * SLOT_BYTES further (the address field counts 16 bytes)
        uint64_t desc_q[NH], desc_slot_k[NH], desc_p[2][S::KB];
        constexpr uint64_t slot_step = S::SLOT_BYTES >> 4;
        for (int h = 0; h < NH; ++h) {
            desc_q[h] = smem_desc(smem_u32(q_buf + h * (kPlQ * 128)));
            desc_slot_k[h] = smem_desc(smem_u32(s.slot[0][h]));
        }
        const uint64_t desc_slot_v = smem_desc_mn(smem_u32(s.slot[0][0]), static_cast<uint32_t>(S::SLOT_HALF));
        for (int part = 0; part < 2; ++part)
            for (int b = 0; b < S::KB; ++b) desc_p[part][b] = smem_desc(smem_u32((part ? p_rest : p_head) + b * (kPlQ * 128)));
        int g = 0, sl = 0, sp = 0, pvc = 0;                          // plane load, its buffer, score plane, P.V plane counters
        uint32_t full_parity = 0;                                    // of bar_full[sl] for load g
        for (int it = 0; it < my_tiles; ++it) {
            if (lane == 0) {
                // ---- pass 1: S_plane = Q . K_plane^T
                for (int pl = 0; pl < RT; ++pl, ++g, ++sp) {
                    bool ready = wait(&s.bar_full[sl], full_parity, 14);
                    if (ready && pl == 0) ready = wait(&s.bar_q, static_cast<uint32_t>(it & 1), 15);
                    // the workers have taken plane sp - 2 out of this score buffer
                    if (ready && sp >= 2) ready = wait(&s.bar_s_free[sp & 1], static_cast<uint32_t>(((sp >> 1) - 1) & 1), 16);
                    if (ready) {
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t d_tmem = tmem + ((sp & 1) ? S::S1 : S::S0);
#pragma unroll
                        for (int h = 0; h < NH; ++h)
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                umma_bf16(d_tmem, desc_q[h] + 2 * kk, desc_slot_k[h] + sl * slot_step + 2 * kk, idesc_s, (h | kk) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&s.bar_s[sp & 1]));          // arrives at once if nothing was issued
                    umma_commit(smem_u32(&s.bar_slot_free[sl]));
                    if (++sl == NS) { sl = 0; full_parity ^= 1u; }
                }
                // ---- pass 2: O += P_plane . V_plane, the head and the remainder of P as two chains
                for (int pl = 0; pl < RT; ++pl, ++g, ++pvc) {
                    bool ready = wait(&s.bar_full[sl], full_parity, 18);
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        if (ready) ready = wait(&s.bar_p_full[part], static_cast<uint32_t>(pvc & 1), 19);
                        if (ready) {
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                            for (int ks = 0; ks < PSP / 16; ++ks)
                                umma_bf16(tmem, desc_p[part][ks >> 2] + 2 * (ks & 3), desc_slot_v + sl * slot_step + 128 * ks, idesc_pv,
                                          (pl | part | ks) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&s.bar_p_free[part]));
                    }
                    umma_commit(smem_u32(&s.bar_slot_free[sl]));
                    if (pl == RT - 1) umma_commit(smem_u32(&s.bar_o));
                    if (++sl == NS) { sl = 0; full_parity ^= 1u; }
                }
            }
            // the workers' epilogue reads O; the next tile's first P.V chain starts beyond the barrier below
            __syncwarp();
            if (tile_barrier_or(*abort_flag != 0u)) break;           // the same decision in every thread
        }
    } else {
        // ==================================================================== workers
        const int lt = warp & 3, half = warp >> 2;                    // query plane of the tile; which thread of the pair
        const int ly = lane >> 3, lx = lane & 7;                      // box order of the Q load: x fastest, then y, then t
        const int r = lt * 32 + lane;                                 // query row of the tile = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>(lt * 32) << 16;
        const uint32_t row_off = static_cast<uint32_t>(r) * 128u, rx = static_cast<uint32_t>(r & 7);
        float* stage = reinterpret_cast<float*>(s.work);             // [column][query]
        const float lscale = rsqrtf(static_cast<float>(D)) * kLog2e;
        // Where this thread's window cells sit is the same for every plane and every tile: kept in
        // registers when the window is small enough, recomputed otherwise.
        constexpr bool kCacheCells = VH * KW <= 16;
        uint32_t cell_stage[kCacheCells ? VH : 1][kCacheCells ? KW : 1];   // element of `stage` holding the cell's score
        uint32_t cell_p[kCacheCells ? VH : 1][kCacheCells ? KW : 1];       // byte offset of the cell inside a P matrix
        auto stage_index = [&](int vv, int ww) { return static_cast<uint32_t>((ly + vv) * RX + lx + ww) * kPlQ + r; };
        auto p_offset = [&](int vv, int ww) {
            const uint32_t col = static_cast<uint32_t>((ly + vv) * RX + lx + ww);
            return (col >> 6) * (kPlQ * 128) + row_off + ((((col & 63) >> 3) ^ rx) << 4) + (col & 7) * 2;
        };
        // The cells of one kernel row are KW neighbouring columns of the query's row of P: they are written as
        // whole 16-byte chunks of 8 columns (one chunk, or two when the cells straddle a chunk boundary).  The
        // other columns of those chunks belong to no cell of this query - the neighbouring kernel rows lie
        // 8 + KW - 1 columns away - so writing them as zeros is right.  Per kernel row, the same for every
        // plane and tile: bits 0-11 / 12-23 the byte offsets of the two chunks (in 16-byte units), bits 24-26
        // the columns by which the cells are shifted inside them.
        // Used for the box of learned offsets (forward 9.95 -> 7.42 ms on the sweep grid: its weights come from
        // shared memory and were read once per matrix).  The fixed windows keep writing their cells one by one:
        // (3,5,5) has its cell offsets in registers and measured 4 % slower this way, (3,7,7) has no registers
        // left for it (84 window scores per thread; a block of this size gets 168 registers per thread).
        constexpr bool kChunkStores = BOUNDED && VH <= 3;
        static_assert(!kChunkStores || (S::P_BYTES <= 65536 && KW <= 7 && RX >= KW + 7),
                      "chunk offsets in 12 bits; a kernel row's chunks touch no other row's cells");
        uint32_t row_geo[VH];
#pragma unroll
        for (int vi = 0; vi < VH; ++vi) {
            const int vv = vi + half * VH < KH ? vi + half * VH : 0;
            const uint32_t col0 = static_cast<uint32_t>((ly + vv) * RX + lx);
            auto chunk_off = [&](uint32_t col) { return (col >> 6) * (kPlQ * 128) + row_off + ((((col & 63) >> 3) ^ rx) << 4); };
            row_geo[vi] = (chunk_off(col0) >> 4) | ((chunk_off(col0 + 8) >> 4) << 12) | ((col0 & 7u) << 24);
        }
        // KW cells (a word each: bf16 head | bf16 remainder << 16) moved to their places among the 16 columns of
        // the row's two chunks by one network of selects, then parted into the words of the head matrix and of
        // the remainder matrix (two columns per word)
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
        if constexpr (kCacheCells) {
#pragma unroll
            for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                for (int ww = 0; ww < KW; ++ww) {
                    const int vv = vi + half * VH < KH ? vi + half * VH : 0;
                    cell_stage[vi][ww] = stage_index(vv, ww);
                    cell_p[vi][ww] = p_offset(vv, ww);
                }
        }
        for (int it = 0; it < my_tiles; ++it) {
            int m, t0, y0, x0;
            locate(static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x), m, t0, y0, x0);
            const int sp0 = it * RT;
            float sc[BOUNDED ? 1 : KT][BOUNDED ? 1 : VH][BOUNDED ? 1 : KW];     // fixed window: this thread's window scores
            if constexpr (!BOUNDED) {
#pragma unroll
                for (int u = 0; u < KT; ++u)
#pragma unroll
                    for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                        for (int ww = 0; ww < KW; ++ww) sc[u][vi][ww] = -INFINITY;
            }

            // BOUNDED: this thread's samples are every other one of the window; their offsets are requested now,
            // so that they have arrived by the time pass 1 is over
            constexpr int WT = BOUNDED ? KT - 2 : 1, WH = BOUNDED ? KH - 2 : 1, WW = BOUNDED ? KW - 2 : 1;
            constexpr int NP = WT * WH * WW, PH = (NP + 1) / 2;
            const int qt = t0 + lt, qy = y0 + ly, qx = x0 + lx;
            const bool in_grid = qt < T && qy < H && qx < W;
            const long long n = (static_cast<long long>(qt) * H + qy) * W + qx;
            float offv[BOUNDED ? PH : 1][3];
            if constexpr (BOUNDED) {
                const float* off_row = offsets + (n * heads + m) * (NP * 3);
#pragma unroll
                for (int i = 0; i < PH; ++i) {
                    const int p = 2 * i + half;
                    offv[i][0] = offv[i][1] = offv[i][2] = 0.0f;
                    if (in_grid && p < NP) {
                        offv[i][0] = __ldg(off_row + p * 3); offv[i][1] = __ldg(off_row + p * 3 + 1); offv[i][2] = __ldg(off_row + p * 3 + 2);
                    }
                }
            }

            // ---------------------------------------------------------- pass 1: the window's scores, plane by plane
            for (int pl = 0; pl < RT; ++pl) {
                const int sp = sp0 + pl;
                wait(&s.bar_s[sp & 1], static_cast<uint32_t>((sp >> 1) & 1), 21);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int u_rt = pl - lt;                             // the kernel plane this region plane is to the warp's queries
                if (u_rt >= 0 && u_rt < KT) {
                    const uint32_t sbuf = tmem + lane_base + ((sp & 1) ? S::S1 : S::S0);
                    for (int piece = half; piece < S::PIECES; piece += 2) {
                        uint32_t regs[32];
                        tmem_load_32(sbuf + piece * 32, regs);
#pragma unroll
                        for (int i = 0; i < 32; ++i) stage[(piece * 32 + i) * kPlQ + r] = __uint_as_float(regs[i]);
                    }
                    named_barrier_sync(1 + lt, 64);                   // the two warps of this quadrant: plane staged
                    if constexpr (BOUNDED) {
                        // the box lives in shared memory: the plane's index may stay a run-time value (one copy of
                        // the code instead of one per kernel plane)
#pragma unroll
                        for (int vi = 0; vi < VH; ++vi) {
                            const int vv = vi + half * VH;
                            if (vv >= KH) continue;
#pragma unroll
                            for (int ww = 0; ww < KW; ++ww)
                                s.box[((u_rt * KH + vv) * KW + ww) * kPlQ + r] =
                                    stage[kCacheCells ? cell_stage[kCacheCells ? vi : 0][kCacheCells ? ww : 0] : stage_index(vv, ww)] * lscale;
                        }
                    } else {
#pragma unroll
                        for (int u = 0; u < KT; ++u) {
                            if (u != u_rt) continue;                  // static register indices for sc
#pragma unroll
                            for (int vi = 0; vi < VH; ++vi) {
                                const int vv = vi + half * VH;
                                if (vv >= KH) continue;
#pragma unroll
                                for (int ww = 0; ww < KW; ++ww)
                                    sc[u][vi][ww] = stage[kCacheCells ? cell_stage[kCacheCells ? vi : 0][kCacheCells ? ww : 0] : stage_index(vv, ww)] * lscale;
                            }
                        }
                    }
                    named_barrier_sync(1 + lt, 64);                   // both have picked: the staging rows may be refilled
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s.bar_s_free[sp & 1]));
            }

            float mx, sum, inv;
            if constexpr (BOUNDED) {
                // ------------------------------------------------------ learned offsets below 1 in size: the eight corners
                // of every sample lie in the query's box, whose scores are in shared memory.  The two threads of
                // a query take every other sample: logit = trilinear combination of the corner scores (positions
                // outside the grid hold 0: the zero-padded key), softmax, then the weights alpha_p * w_c are summed
                // into the box cells in place of the scores.
                named_barrier_sync(1 + lt, 64);                       // the whole box is in place
                float lg[PH], fr[PH][3];
                int cellv[PH];
                // position of a sample relative to the box origin, exactly as the general kernel forms it:
                // float(coord + b) + offset, floor, difference - all in fp32
#pragma unroll
                for (int i = 0; i < PH; ++i) {
                    const int p = 2 * i + half;
                    const int w = p % WW, v = (p / WW) % WH, u = p / (WW * WH);
                    const float pt = __fadd_rn(static_cast<float>(qt + u - WT / 2), offv[i][0]),
                                py = __fadd_rn(static_cast<float>(qy + v - WH / 2), offv[i][1]),
                                px = __fadd_rn(static_cast<float>(qx + w - WW / 2), offv[i][2]);
                    const float flt = floorf(pt), fly = floorf(py), flx = floorf(px);
                    float ft = __fsub_rn(pt, flt), fy = __fsub_rn(py, fly), fx = __fsub_rn(px, flx);
                    // cell index of corner (0,0,0) inside the box (origin = query - K/2).  An offset just below +1
                    // can round the fp32 position up to the next integer: the sample then sits exactly on the
                    // box's last position, which is written as the cell before it with fraction 1.  (The clamps
                    // also keep a garbage offset from indexing outside the box.)
                    int ct = max(static_cast<int>(flt) - (qt - KT / 2), 0), cy = max(static_cast<int>(fly) - (qy - KH / 2), 0),
                        cx = max(static_cast<int>(flx) - (qx - KW / 2), 0);
                    if (ct > KT - 2) { ct = KT - 2; ft = 1.0f; }
                    if (cy > KH - 2) { cy = KH - 2; fy = 1.0f; }
                    if (cx > KW - 2) { cx = KW - 2; fx = 1.0f; }
                    cellv[i] = ((ct * KH + cy) * KW + cx) * kPlQ + r;
                    fr[i][0] = ft; fr[i][1] = fy; fr[i][2] = fx;
                }
                mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < PH; ++i) {
                    const int p = 2 * i + half;
                    lg[i] = -INFINITY;
                    if (p < NP) {
                        const float ft = fr[i][0], fy = fr[i][1], fx = fr[i][2];
                        const float* bx = s.box + cellv[i];
                        float a[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) a[c] = bx[(((c >> 2) * KH + ((c >> 1) & 1)) * KW + (c & 1)) * kPlQ];
                        const float x0v = fmaf(fx, a[1] - a[0], a[0]), x1v = fmaf(fx, a[3] - a[2], a[2]);
                        const float x2v = fmaf(fx, a[5] - a[4], a[4]), x3v = fmaf(fx, a[7] - a[6], a[6]);
                        const float y0v = fmaf(fy, x1v - x0v, x0v), y1v = fmaf(fy, x3v - x2v, x2v);
                        lg[i] = fmaf(ft, y1v - y0v, y0v);
                        mx = fmaxf(mx, lg[i]);
                    }
                }
                s.pair_max[tid] = mx;
                named_barrier_sync(1 + lt, 64);
                mx = fmaxf(mx, s.pair_max[tid ^ 128]);
                sum = 0.0f;
#pragma unroll
                for (int i = 0; i < PH; ++i) { lg[i] = exp2f(lg[i] - mx); sum += lg[i]; }
                s.pair_sum[tid] = sum;
                named_barrier_sync(1 + lt, 64);                       // also: every score of the box has been read
                sum += s.pair_sum[tid ^ 128];
                inv = 1.0f / sum;
                // the box now collects the weights: cleared (each thread its rows), then the two threads add
                // their samples one after the other (plain read-add-write: no two threads at a cell at once)
#pragma unroll
                for (int u = 0; u < KT; ++u)
#pragma unroll
                    for (int vi = 0; vi < VH; ++vi) {
                        const int vv = vi + half * VH;
                        if (vv >= KH) continue;
#pragma unroll
                        for (int ww = 0; ww < KW; ++ww) s.box[((u * KH + vv) * KW + ww) * kPlQ + r] = 0.0f;
                    }
                named_barrier_sync(1 + lt, 64);
#pragma unroll
                for (int turn = 0; turn < 2; ++turn) {
                    if (turn == half) {
#pragma unroll
                        for (int i = 0; i < PH; ++i) {
                            const int p = 2 * i + half;
                            if (p >= NP) continue;
                            const float ft = fr[i][0], fy = fr[i][1], fx = fr[i][2];
                            float* bx = s.box + cellv[i];
                            const float al = lg[i] * inv;
                            const float wt[2] = {1.0f - ft, ft}, wy[2] = {1.0f - fy, fy}, wx[2] = {1.0f - fx, fx};
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                bx[(((c >> 2) * KH + ((c >> 1) & 1)) * KW + (c & 1)) * kPlQ] += al * (wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1]);
                        }
                    }
                    named_barrier_sync(1 + lt, 64);
                }
            } else {
                // ------------------------------------------------------ softmax over the window (two threads per query)
                mx = -INFINITY;
    #pragma unroll
                for (int u = 0; u < KT; ++u)
    #pragma unroll
                    for (int vi = 0; vi < VH; ++vi)
    #pragma unroll
                        for (int ww = 0; ww < KW; ++ww) mx = fmaxf(mx, sc[u][vi][ww]);
                s.pair_max[tid] = mx;
                named_barrier_sync(1 + lt, 64);
                mx = fmaxf(mx, s.pair_max[tid ^ 128]);
                sum = 0.0f;
    #pragma unroll
                for (int u = 0; u < KT; ++u)
    #pragma unroll
                    for (int vi = 0; vi < VH; ++vi)
    #pragma unroll
                        for (int ww = 0; ww < KW; ++ww) {
                            sc[u][vi][ww] = exp2f(sc[u][vi][ww] - mx);        // cells this thread does not own: exp2(-inf) = 0
                            sum += sc[u][vi][ww];
                        }
                s.pair_sum[tid] = sum;
                named_barrier_sync(1 + lt, 64);
                sum += s.pair_sum[tid ^ 128];
                inv = 1.0f / sum;
            }
            if (half == 0 && in_grid) lse[n * heads + m] = (mx + log2f(sum)) * kLn2;

            // ---------------------------------------------------------- pass 2: this query's row of P, plane by plane
            // A thread's cells sit at the same columns of P in each of its KT planes: the row is cleared
            // once per tile (the area held scores), the cells are overwritten plane after plane and
            // written as zeros for the plane after the last.
            for (int pl = 0; pl < RT; ++pl) {
                const int pvc = it * RT + pl;
                const int u_rt = pl - lt;
                const bool mine = u_rt >= 0 && u_rt < KT;
                if (pl == 0) {
                    // the chains of the previous tile have run (its epilogue waited for them); all staging
                    // reads of this tile are done once every worker is here
                    named_barrier_sync(5, kPlWorkers);
                    unsigned char* dst = (half ? p_rest : p_head) + row_off;
#pragma unroll
                    for (int c = 0; c < PSP / 8; ++c)
                        *reinterpret_cast<uint4*>(dst + (c >> 3) * (kPlQ * 128) + (((c & 7) ^ rx) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                    named_barrier_sync(1 + lt, 64);                   // both matrices of the row are clear before cells land
                }
                if constexpr (kChunkStores) {
                    // The words of kernel row vi of this plane for the head and the remainder matrix.  With few rows per
                    // thread the remainder words wait in registers while the head matrix goes out; with four rows
                    // (the (3,7,7) window: 84 window scores live in registers already) they are formed again.
                    constexpr bool kKeepRest = VH <= 3;
                    auto row_words = [&](auto vi_c, uint32_t (&head)[8], uint32_t (&rest)[8]) {
                        constexpr int vi = decltype(vi_c)::value;         // a constant, so that sc[][vi][] stays in registers
                        const int vv = vi + half * VH;
                        uint32_t cell[8];
#pragma unroll
                        for (int ww = 0; ww < 8; ++ww) cell[ww] = 0u;
                        auto split = [](float p) {
                            const __nv_bfloat16 hd = __float2bfloat16_rn(p);
                            const __nv_bfloat16 rm = __float2bfloat16_rn(p - __bfloat162float(hd));
                            return static_cast<uint32_t>(__bfloat16_as_ushort(hd)) | (static_cast<uint32_t>(__bfloat16_as_ushort(rm)) << 16);
                        };
                        if constexpr (BOUNDED) {
                            if (u_rt < KT) {
#pragma unroll
                                for (int ww = 0; ww < KW; ++ww) cell[ww] = split(s.box[((u_rt * KH + vv) * KW + ww) * kPlQ + r]);
                            }
                        } else {
#pragma unroll
                            for (int u = 0; u < KT; ++u) {
                                if (u != u_rt) continue;
#pragma unroll
                                for (int ww = 0; ww < KW; ++ww) cell[ww] = split(sc[u][vi][ww] * inv);
                            }
                        }
                        align_row(row_geo[vi], cell, head, rest);
                    };
                    uint32_t kept[kKeepRest ? VH : 1][8];
                    const bool writes = mine || u_rt == KT;               // u_rt == KT: the cells go back to zero
                    if (pl > 0) wait(&s.bar_p_free[0], static_cast<uint32_t>((pvc - 1) & 1), 22);   // the head chain of the plane before
                    // f(constant) for every kernel row of this thread
                    auto for_rows = [&](auto&& f) {
                        f(std::integral_constant<int, 0>{});
                        if constexpr (VH > 1) f(std::integral_constant<int, 1>{});
                        if constexpr (VH > 2) f(std::integral_constant<int, 2>{});
                        if constexpr (VH > 3) f(std::integral_constant<int, 3>{});
                        static_assert(VH <= 4, "kernel rows per thread");
                    };
                    if (writes) {
                        for_rows([&](auto vi_c) {
                            constexpr int vi = decltype(vi_c)::value;
                            if (vi + half * VH >= KH) return;
                            uint32_t head[8], rest[8];
                            row_words(vi_c, head, rest);
                            store_chunks(p_head, row_geo[vi], head);
                            if constexpr (kKeepRest) {
#pragma unroll
                                for (int j = 0; j < 8; ++j) kept[vi][j] = rest[j];
                            }
                        });
                    }
                    fence_async_smem();                                   // the MMAs read P through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s.bar_p_full[0]));
                    if (pl > 0) wait(&s.bar_p_free[1], static_cast<uint32_t>((pvc - 1) & 1), 22);   // the remainder chain of the plane before
                    if (writes) {
                        for_rows([&](auto vi_c) {
                            constexpr int vi = decltype(vi_c)::value;
                            if (vi + half * VH >= KH) return;
                            if constexpr (kKeepRest) {
                                store_chunks(p_rest, row_geo[vi], kept[vi]);
                            } else {
                                uint32_t head[8], rest[8];
                                row_words(vi_c, head, rest);
                                store_chunks(p_rest, row_geo[vi], rest);
                            }
                        });
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s.bar_p_full[1]));
                } else {
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        if (pl > 0) wait(&s.bar_p_free[part], static_cast<uint32_t>((pvc - 1) & 1), 22);   // the chain of the plane before
                        if (mine || u_rt == KT) {
                            unsigned char* dst = part ? p_rest : p_head;
#pragma unroll
                            for (int u = 0; u <= KT; ++u) {
                                if (u != u_rt) continue;
#pragma unroll
                                for (int vi = 0; vi < VH; ++vi) {
                                    const int vv = vi + half * VH;
                                    if (vv >= KH) continue;
#pragma unroll
                                    for (int ww = 0; ww < KW; ++ww) {
                                        float p = 0.0f;
                                        if constexpr (BOUNDED) {
                                            if (u < KT) p = s.box[(((u < KT ? u : 0) * KH + vv) * KW + ww) * kPlQ + r];
                                        } else {
                                            if (u < KT) p = sc[u < KT ? u : 0][vi][ww] * inv;
                                        }
                                        __nv_bfloat16 val = __float2bfloat16_rn(p);
                                        if (part) val = __float2bfloat16_rn(p - __bfloat162float(val));
                                        *reinterpret_cast<__nv_bfloat16*>(dst + (kCacheCells ? cell_p[kCacheCells ? vi : 0][kCacheCells ? ww : 0] : p_offset(vv, ww))) = val;
                                    }
                                }
                            }
                        }
                        fence_async_smem();                               // the MMAs read P through the async proxy
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&s.bar_p_full[part]));
                    }
                }
            }

            // ---------------------------------------------------------- epilogue: the pair splits the channels
            wait(&s.bar_o, static_cast<uint32_t>(it & 1), 23);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            {
                constexpr int CH = D / 2;                             // channels per thread of the pair
#pragma unroll
                for (int c0 = 0; c0 < CH; c0 += 32) {
                    uint32_t regs[32];
                    tmem_load_32(tmem + lane_base + half * CH + c0, regs);
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
            if (tile_barrier_or(*abort_flag != 0u)) break;           // O is free for the next tile's chains
        }
    }
    // Gave up: loads may still be in flight towards this CTA's shared memory; give them a bounded time.
    if (*abort_flag && tid == kPlWorkers) {
        for (int i = 0; i < NS; ++i) {
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 0u, 1u << 16);
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 1u, 1u << 16);
        }
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

template <int D, int KT, int KH, int KW, bool BOUNDED>
cudaError_t launch_planes(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, void* out, float* lse,
                          const Problem& pr, int* flag, const float* offsets, const int* gate, cudaStream_t stream) {
    const int tiles_x = (pr.W + kPlTX - 1) / kPlTX, tiles_y = (pr.H + kPlTY - 1) / kPlTY,
              tiles_t = (pr.T + kPlTT - 1) / kPlTT;
    const size_t smem = sizeof(PlSmem<D, KT, KH, KW, BOUNDED>) + 1024;
    auto kern = fixed_window_planes_kernel<D, KT, KH, KW, BOUNDED>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    if (total * (2 * (kPlTT + KT - 1)) >= (1LL << 31)) return cudaErrorInvalidValue;   // the kernel counts planes in 32 bits
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kPlThreads, smem, stream>>>(mq, mk, mv, static_cast<__nv_bfloat16*>(out), lse, pr.T, pr.H, pr.W, pr.heads,
                                             tiles_x, tiles_y, static_cast<int>(total), flag, offsets, gate);
    return cudaGetLastError();
}

// *gate = 1 if some offset component is NaN, infinite or not below 1 in size (plain stores of the same
// value: no ordering needed).  The caller has set *gate = 0 on the same stream.
__global__ void __launch_bounds__(256)
offsets_bound_kernel(const float4* __restrict__ off4, long long count4, const float* __restrict__ tail, int tail_count,
                     int* __restrict__ gate) {
    bool bad = false;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < count4; i += stride) {
        const float4 o = __ldg(off4 + i);
        bad = bad || !(fabsf(o.x) < 1.0f) || !(fabsf(o.y) < 1.0f) || !(fabsf(o.z) < 1.0f) || !(fabsf(o.w) < 1.0f);
    }
    if (blockIdx.x == 0 && static_cast<int>(threadIdx.x) < tail_count) bad = bad || !(fabsf(tail[threadIdx.x]) < 1.0f);
    if (__syncthreads_or(bad) && threadIdx.x == 0) *gate = 1;
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
    if (tiles * pr.heads * 2 * (kPlTT + pr.kt - 1) >= (1LL << 31)) return false;     // the kernel counts planes in 32 bits
    int* flag = timeout_flag_device_address();
    CUtensorMap mq, mk, mv;
    if (!flag || !make_plane_maps(q, k, v, pr, pr.kh, pr.kw, &mq, &mk, &mv)) return false;
    if (pr.d == 128)
        *err = w355 ? launch_planes<128, 3, 5, 5, false>(mq, mk, mv, out, lse, pr, flag, nullptr, nullptr, stream)
                    : launch_planes<128, 3, 7, 7, false>(mq, mk, mv, out, lse, pr, flag, nullptr, nullptr, stream);
    else
        *err = w355 ? launch_planes<64, 3, 5, 5, false>(mq, mk, mv, out, lse, pr, flag, nullptr, nullptr, stream)
                    : launch_planes<64, 3, 7, 7, false>(mq, mk, mv, out, lse, pr, flag, nullptr, nullptr, stream);
    return true;
}

bool bounded_offsets_shape_covered(const Problem& pr, bool bf16) {
    return bf16 && (pr.d == 128 || pr.d == 64) && pr.kt == 3 && pr.kh == 3 && pr.kw == 3;
}

cudaError_t launch_offsets_bound_check(const float* offsets, long long count, int* gate, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(gate, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    const long long count4 = count / 4;
    long long blocks = (count4 + 255) / 256;
    if (blocks > 148LL * 8) blocks = 148LL * 8;
    if (blocks < 1) blocks = 1;
    offsets_bound_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(offsets), count4, offsets + count4 * 4, static_cast<int>(count - count4 * 4), gate);
    return cudaGetLastError();
}

bool try_bounded_offsets_forward(const void* q, const void* k, const void* v, const float* offsets, const int* gate,
                                 void* out, float* lse, const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (!bounded_offsets_shape_covered(pr, true)) return false;
    const long long tiles = static_cast<long long>((pr.W + kPlTX - 1) / kPlTX) * ((pr.H + kPlTY - 1) / kPlTY) *
                            ((pr.T + kPlTT - 1) / kPlTT);
    if (tiles * pr.heads * 2 * (kPlTT + pr.kt + 2 - 1) >= (1LL << 31)) return false;
    int* flag = timeout_flag_device_address();
    CUtensorMap mq, mk, mv;
    if (!flag || !make_plane_maps(q, k, v, pr, pr.kh + 2, pr.kw + 2, &mq, &mk, &mv)) return false;
    *err = pr.d == 128 ? launch_planes<128, 5, 5, 5, true>(mq, mk, mv, out, lse, pr, flag, offsets, gate, stream)
                       : launch_planes<64, 5, 5, 5, true>(mq, mk, mv, out, lse, pr, flag, offsets, gate, stream);
    return true;
}

}  // namespace dsa3d
