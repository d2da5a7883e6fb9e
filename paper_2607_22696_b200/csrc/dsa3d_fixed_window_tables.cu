// Dot-product tables of the fixed-window backward on the tensor cores.
//
// With zero offsets the backward of a query needs  a_j = q . K_j  and  b_j = dO . V_j  for the key
// positions j of its window and of the window's +1 neighbours along each axis (the one-sided
// derivative of the trilinear weights at an integer position): the box of (kt+1)(kh+1)(kw+1)
// positions whose first corner is query - (kt/2, kh/2, kw/2).  For a tile of 4 x 4 x 8 queries
// these are entries of the dense products  Q_tile . K_region^T  and  dO_tile . V_region^T  over the
// tile's region (tile + box - 1 per axis), which this kernel forms by tcgen05.mma one region
// plane at a time (fp32 accumulators in TMEM) and from which every thread copies the box of its
// query into a table in global memory:  table[item][0][cell] = a,  table[item][1][cell] = b  with
// item = token * heads + head and cell = (u * (kh+1) + v) * (kw+1) + w.  Positions outside the grid
// read as zero rows (TMA fill), i.e. a = b = 0, which is what the gather kernel would have used.
// fixed_window_backward_query_kernel then takes its dot products from the table instead of
// gathering K and V rows.
//
// Roles as in the plane-by-plane forward: 8 worker warps copy scores (the two warps that share a TMEM
// quadrant split a plane's columns and the box's rows along y between them), one more warp holds the
// thread that issues the TMA loads, two more one thread each that issues the MMAs of every other plane;
// mbarriers order them, every wait is bounded, and a wait that runs out raises the library's timeout
// flag, after which nobody waits any more.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kTbTT = 4, kTbTY = 4, kTbTX = 8, kTbQ = kTbTT * kTbTY * kTbTX;    // 128 queries per tile
constexpr int kTbSplit = 2;                                                   // worker warps per TMEM quadrant
constexpr int kTbWorkers = 128 * kTbSplit, kTbThreads = kTbWorkers + 96;      // + loading warp + two MMA warps
constexpr int kTbSlots = 4;                                                   // plane buffers, at most
constexpr int kTbScoreBufs = 4;                                               // score planes in flight in TMEM, at most

template <int D, int KT, int KH, int KW>
struct TableShape {
    static constexpr int NH = D / 64;
    static constexpr int BT = KT + 1, BY = KH + 1, BX = KW + 1;     // the box of a query
    static constexpr int CELLS = BT * BY * BX, CELLS8 = (CELLS + 7) / 8 * 8;
    static constexpr int RT = kTbTT + BT - 1, RY = kTbTY + BY - 1, RX = kTbTX + BX - 1;
    static constexpr int PS = RY * RX, PSP = (PS + 15) / 16 * 16;
    static constexpr int PIECES = (PS + 31) / 32;
    static constexpr int VH = (BY + kTbSplit - 1) / kTbSplit;        // consecutive box rows along y per thread of a query's group
    static constexpr int SBUF = PIECES * 32;
    static constexpr int SLOT_HALF = PSP * 128;
    // a large score plane is staged and picked from in two halves of its columns
    static constexpr int SUBS = PIECES > 4 ? 2 : 1, PPS = (PIECES + SUBS - 1) / SUBS;
    static constexpr int STAGE_BYTES = PPS * 32 * kTbQ * 4;
    static constexpr int A_BYTES = NH * kTbQ * 128;                 // Q or dO rows of the tile
    static constexpr int SLOT_BYTES = NH * ((SLOT_HALF + 1023) / 1024 * 1024);
    // as many score planes in TMEM and plane buffers in shared memory as fit, up to four each
    static constexpr int NB = 512 / SBUF < kTbScoreBufs ? 512 / SBUF : kTbScoreBufs;
    static constexpr int NS_FIT = (227 * 1024 - 4096 - 2 * A_BYTES - STAGE_BYTES) / SLOT_BYTES;
    static constexpr int NS = NS_FIT > kTbSlots ? kTbSlots : NS_FIT;
    static_assert(PSP <= 256 && NB >= 2 && NS >= 2, "plane too large");
    static_assert(SLOT_HALF % 1024 == 0 || PSP % 8 == 0, "");
};

template <int D, int KT, int KH, int KW>
struct __align__(1024) TbSmem {
    using S = TableShape<D, KT, KH, KW>;
    unsigned char a[2][S::A_BYTES];                                 // Q, dO: 64-channel halves, swizzled 128-byte rows
    unsigned char slot[S::NS][S::NH][(S::SLOT_HALF + 1023) / 1024 * 1024];
    unsigned char stage[S::STAGE_BYTES];                            // a score plane as [column][query] floats
    uint64_t bar_a[2], bar_full[kTbSlots], bar_slot_free[kTbSlots], bar_s[kTbScoreBufs], bar_s_free[kTbScoreBufs];
    uint32_t tmem_base;
    uint32_t abort;
};

// the warps that share a TMEM quadrant
__device__ __forceinline__ void pair_barrier(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(32 * kTbSplit) : "memory"); }

template <int D, int KT, int KH, int KW>
__global__ void __launch_bounds__(kTbThreads, 1)
fixed_window_tables_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_do,
                           const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                           float* __restrict__ table, int T, int H, int W, int heads, int tiles_x, int tiles_y, int total,
                           int* timeout_flag, const int* __restrict__ gate) {
    using S = TableShape<D, KT, KH, KW>;
    constexpr int NH = S::NH, RT = S::RT, RX = S::RX, PS = S::PS, PSP = S::PSP, VH = S::VH, NS = S::NS;
    constexpr int BT = S::BT, BY = S::BY, BX = S::BX;
    constexpr int JOBS = 2 * RT;                                      // per tile: RT planes of K (against Q), RT of V (against dO)
    constexpr int NB = S::NB;
    constexpr int TMEM_COLS = NB * S::SBUF <= 128 ? 128 : (NB * S::SBUF <= 256 ? 256 : 512);
    extern __shared__ unsigned char raw[];
    TbSmem<D, KT, KH, KW>& s =
        *reinterpret_cast<TbSmem<D, KT, KH, KW>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&s.bar_a[i]), 1);
        for (int i = 0; i < NB; ++i) {
            mbar_init(smem_u32(&s.bar_s[i]), 1);
            mbar_init(smem_u32(&s.bar_s_free[i]), kTbWorkers / 32);
        }
        for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&s.bar_full[i]), 1); mbar_init(smem_u32(&s.bar_slot_free[i]), 1); }
        s.abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
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
    const int tiles_per_head = total / heads;
    auto locate = [&](int item, int& m, int& t0, int& y0, int& x0) {
        m = item / tiles_per_head;
        int tile = item - m * tiles_per_head;
        x0 = (tile % tiles_x) * kTbTX; tile /= tiles_x;
        y0 = (tile % tiles_y) * kTbTY;
        t0 = (tile / tiles_y) * kTbTT;
    };
    // behind a check of learned offsets: nothing to do unless the check left 0 in *gate
    const bool open = gate == nullptr || *gate == 0;
    const int my_tiles = open && static_cast<int>(blockIdx.x) < total
                             ? (total - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;
    auto tile_item = [&](int ti) { return static_cast<int>(blockIdx.x) + ti * static_cast<int>(gridDim.x); };

    if (warp == kTbWorkers / 32) {
        // ==================================================================== loading thread
        if (lane == 0 && my_tiles > 0) {
            const int jobs_total = my_tiles * JOBS;
            auto load_a = [&](int which, int ti) {                    // Q (0) or dO (1) rows of tile ti
                int m, t0, y0, x0;
                locate(tile_item(ti), m, t0, y0, x0);
                mbar_expect_tx(smem_u32(&s.bar_a[which]), static_cast<uint32_t>(S::A_BYTES));
                for (int h = 0; h < NH; ++h)
                    tma_load_5d(smem_u32(s.a[which] + h * (kTbQ * 128)), which ? &map_do : &map_q, smem_u32(&s.bar_a[which]),
                                h * 64, m, x0, y0, t0);
            };
            int tile_index = 0, j = 0, m, t0, y0, x0;
            locate(tile_item(0), m, t0, y0, x0);
            load_a(0, 0);
            load_a(1, 0);
            for (int g = 0; g < jobs_total; ++g) {
                const int sl = g % NS;
                if (g >= NS) {
                    if (!wait(&s.bar_slot_free[sl], static_cast<uint32_t>((g / NS - 1) & 1), 24)) break;
                    // the MMAs of plane load g - NS have run: after a tile's last K plane its Q rows are free,
                    // after its last V plane its dO rows
                    const int done = g - NS, done_tile = done / JOBS, dj = done - done_tile * JOBS;
                    if (done_tile + 1 < my_tiles) {
                        if (dj == RT - 1) load_a(0, done_tile + 1);
                        if (dj == JOBS - 1) load_a(1, done_tile + 1);
                    }
                }
                const uint32_t bar = smem_u32(&s.bar_full[sl]);
                mbar_expect_tx(bar, static_cast<uint32_t>(NH) * PS * 128u);
                const CUtensorMap* map = j < RT ? &map_k : &map_v;
                const int plane = j < RT ? j : j - RT;
                for (int h = 0; h < NH; ++h)
                    tma_load_5d(smem_u32(s.slot[sl][h]), map, bar, h * 64, m, x0 - KW / 2, y0 - KH / 2, t0 - KT / 2 + plane);
                if (++j == JOBS) {
                    j = 0;
                    if (++tile_index < my_tiles) locate(tile_item(tile_index), m, t0, y0, x0);
                }
            }
        }
    } else if (warp >= kTbWorkers / 32 + 1) {
        // ==================================================================== two MMA threads
        // Issuing a tcgen05.mma costs its thread some tens of cycles whatever the size of the product, and a
        // region plane is a small product (N = PSP), so two threads share the planes: thread `mt` takes the
        // planes with number = mt (mod 2).  (Plane number g = plane load g here; score buffer g mod NB.)
        if (lane == 0) {
            const int mt = warp - (kTbWorkers / 32 + 1);
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kTbQ >> 4) << 24) |
                                       (static_cast<uint32_t>(PSP >> 3) << 17);
            constexpr uint64_t slot_step = sizeof(s.slot[0]) >> 4;
            uint64_t desc_a[2][NH], desc_slot[NH];
            for (int h = 0; h < NH; ++h) {
                desc_a[0][h] = smem_desc(smem_u32(s.a[0] + h * (kTbQ * 128)));
                desc_a[1][h] = smem_desc(smem_u32(s.a[1] + h * (kTbQ * 128)));
                desc_slot[h] = smem_desc(smem_u32(s.slot[0][h]));
            }
            const int jobs_total = my_tiles * JOBS;
            int it = 0, j = mt;                                      // tile and plane load within it of plane g
            for (int g = mt; g < jobs_total; g += 2) {
                const int sl = g % NS, which = j >= RT ? 1 : 0;
                bool ready = wait(&s.bar_full[sl], static_cast<uint32_t>((g / NS) & 1), 25);
                if (ready) ready = wait(&s.bar_a[which], static_cast<uint32_t>(it & 1), 26);
                // the workers have taken plane g - NB out of this score buffer
                if (ready && g >= NB) ready = wait(&s.bar_s_free[g % NB], static_cast<uint32_t>((g / NB - 1) & 1), 27);
                if (ready) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d_tmem = tmem + (g % NB) * S::SBUF;
#pragma unroll
                    for (int h = 0; h < NH; ++h)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_bf16(d_tmem, (which ? desc_a[1][h] : desc_a[0][h]) + 2 * kk, desc_slot[h] + sl * slot_step + 2 * kk,
                                      idesc, (h | kk) ? 1u : 0u);
                }
                umma_commit(smem_u32(&s.bar_s[g % NB]));
                umma_commit(smem_u32(&s.bar_slot_free[sl]));
                j += 2;
                if (j >= JOBS) { j -= JOBS; ++it; }
            }
        }
    } else {
        // ==================================================================== workers
        const int lt = warp & 3, half = warp >> 2;                   // quadrant; which of its kTbSplit warps
        const int ly = lane >> 3, lx = lane & 7;
        const int r = lt * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(lt * 32) << 16;
        float* stage = reinterpret_cast<float*>(s.stage);
        int sp = 0;
        for (int it = 0; it < my_tiles; ++it) {
            int m, t0, y0, x0;
            locate(tile_item(it), m, t0, y0, x0);
            const int qt = t0 + lt, qy = y0 + ly, qx = x0 + lx;
            const bool in_grid = qt < T && qy < H && qx < W;
            const long long item = ((static_cast<long long>(qt) * H + qy) * W + qx) * heads + m;
            float* my_table = table + item * (2 * S::CELLS8);
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                for (int pl = 0; pl < RT; ++pl, ++sp) {
                    if (lane == 0) wait(&s.bar_s[sp % NB], static_cast<uint32_t>((sp / NB) & 1), 28);   // one lane polls for its warp
                    __syncwarp();
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const int u_rt = pl - lt;                         // the box plane this region plane is to the warp's queries
                    if (u_rt >= 0 && u_rt < BT) {
                        const uint32_t sbuf = tmem + lane_base + (sp % NB) * S::SBUF;
                        // this thread's rows of the box plane are neighbours (vv = half * VH ...), so its cells
                        // are one contiguous run of the table: written as 16-byte pieces when BX = 4 (a warp's
                        // stores then fill whole 32-byte sectors instead of touching each one eight times)
                        float* dst = my_table + which * S::CELLS8 + u_rt * (BY * BX) + half * VH * BX;
                        float cells[VH * BX];
#pragma unroll
                        for (int i = 0; i < VH * BX; ++i) cells[i] = 0.0f;
#pragma unroll
                        for (int sub = 0; sub < S::SUBS; ++sub) {
                            constexpr int PPS = S::PPS;
                            for (int piece = sub * PPS + half; piece < (sub + 1) * PPS && piece < S::PIECES; piece += kTbSplit) {
                                uint32_t regs[32];
                                tmem_load_32(sbuf + piece * 32, regs);
#pragma unroll
                                for (int i = 0; i < 32; ++i) stage[((piece - sub * PPS) * 32 + i) * kTbQ + r] = __uint_as_float(regs[i]);
                            }
                            pair_barrier(1 + lt);                     // the plane (or this half of its columns) is staged
                            if (in_grid && !*abort_flag) {
#pragma unroll
                                for (int vi = 0; vi < VH; ++vi)
#pragma unroll
                                    for (int ww = 0; ww < BX; ++ww) {
                                        const int vv = vi + half * VH;
                                        const int col = (ly + vv) * RX + lx + ww - sub * PPS * 32;
                                        if (vv < BY && (S::SUBS == 1 || (col >= 0 && col < PPS * 32))) cells[vi * BX + ww] = stage[col * kTbQ + r];
                                    }
                            }
                            pair_barrier(1 + lt);                     // both have copied: the staging rows may be refilled
                        }
                        if (in_grid && !*abort_flag) {
                            // the run of VH * BX floats, in the widest pieces its alignment allows
                            constexpr int RUN = VH * BX;
                            constexpr bool whole = BY % kTbSplit == 0;     // every thread of the group has all VH rows
                            if constexpr (whole && RUN % 4 == 0 && (BY * BX) % 4 == 0 && S::CELLS8 % 4 == 0) {
#pragma unroll
                                for (int i = 0; i < RUN / 4; ++i)
                                    reinterpret_cast<float4*>(dst)[i] = make_float4(cells[4 * i], cells[4 * i + 1], cells[4 * i + 2], cells[4 * i + 3]);
                            } else if constexpr (whole && RUN % 4 == 2 && (BY * BX) % 4 == 0 && S::CELLS8 % 4 == 0) {
                                // the run starts 16-byte aligned for every other thread of the group and 8 bytes
                                // off for the others: one 8-byte piece at the far or the near end, 16-byte pieces between
                                const int lead = (half * RUN) & 3;                  // 0 or 2 floats before the first aligned piece
                                if (lead) *reinterpret_cast<float2*>(dst) = make_float2(cells[0], cells[1]);
#pragma unroll
                                for (int i = 0; i < RUN / 4; ++i) {
                                    float4 piece;
                                    piece.x = lead ? cells[4 * i + 2] : cells[4 * i];
                                    piece.y = lead ? cells[4 * i + 3] : cells[4 * i + 1];
                                    piece.z = lead ? cells[4 * i + 4] : cells[4 * i + 2];
                                    piece.w = lead ? cells[4 * i + 5] : cells[4 * i + 3];
                                    *reinterpret_cast<float4*>(dst + lead + 4 * i) = piece;
                                }
                                if (!lead) *reinterpret_cast<float2*>(dst + RUN - 2) = make_float2(cells[RUN - 2], cells[RUN - 1]);
                            } else if constexpr (whole && RUN % 2 == 0 && (BY * BX) % 2 == 0 && S::CELLS8 % 2 == 0) {
#pragma unroll
                                for (int i = 0; i < RUN / 2; ++i) reinterpret_cast<float2*>(dst)[i] = make_float2(cells[2 * i], cells[2 * i + 1]);
                            } else {
#pragma unroll
                                for (int i = 0; i < VH * BX; ++i)
                                    if (i / BX + half * VH < BY) dst[i] = cells[i];
                            }
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s.bar_s_free[sp % NB]));
                }
            }
        }
    }
    if (*abort_flag && tid == kTbWorkers) {       // gave up: loads may still be on their way into this CTA's shared memory
        for (int i = 0; i < NS; ++i) {
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 0u, 1u << 16);
            mbar_wait_limit(smem_u32(&s.bar_full[i]), 1u, 1u << 16);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_wait_limit(smem_u32(&s.bar_a[i]), 0u, 1u << 16);
            mbar_wait_limit(smem_u32(&s.bar_a[i]), 1u, 1u << 16);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS));
}

template <int D, int KT, int KH, int KW>
cudaError_t launch_tables(const void* q, const void* k, const void* v, const void* dout, float* table, const Problem& pr,
                          int* flag, cudaStream_t stream, bool* unsupported, const int* gate = nullptr) {
    using S = TableShape<D, KT, KH, KW>;
    const unsigned long long d = static_cast<unsigned long long>(pr.d), hd = static_cast<unsigned long long>(pr.heads);
    const unsigned long long dims[5] = {d, hd, static_cast<unsigned long long>(pr.W), static_cast<unsigned long long>(pr.H),
                                        static_cast<unsigned long long>(pr.T)};
    const unsigned long long strides[4] = {d * 2, hd * d * 2, static_cast<unsigned long long>(pr.W) * hd * d * 2,
                                           static_cast<unsigned long long>(pr.H) * pr.W * hd * d * 2};
    const unsigned box_a[5] = {64, 1, kTbTX, kTbTY, kTbTT};
    const unsigned box_p[5] = {64, 1, static_cast<unsigned>(S::RX), static_cast<unsigned>(S::RY), 1};
    CUtensorMap mq, mdo, mk, mv;
    if (!encode_tensor_map_bf16(&mq, q, 5, dims, strides, box_a, true) ||
        !encode_tensor_map_bf16(&mdo, dout, 5, dims, strides, box_a, true) ||
        !encode_tensor_map_bf16(&mk, k, 5, dims, strides, box_p, true) ||
        !encode_tensor_map_bf16(&mv, v, 5, dims, strides, box_p, true)) {
        *unsupported = true;
        return cudaSuccess;
    }
    const int tiles_x = (pr.W + kTbTX - 1) / kTbTX, tiles_y = (pr.H + kTbTY - 1) / kTbTY,
              tiles_t = (pr.T + kTbTT - 1) / kTbTT;
    const long long total = static_cast<long long>(tiles_x) * tiles_y * tiles_t * pr.heads;
    if (total * (2 * S::RT) >= (1LL << 31)) {                          // the kernel counts planes in 32 bits
        *unsupported = true;
        return cudaSuccess;
    }
    const size_t smem = sizeof(TbSmem<D, KT, KH, KW>) + 1024;
    auto kern = fixed_window_tables_kernel<D, KT, KH, KW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kTbThreads, smem, stream>>>(mq, mdo, mk, mv, table, pr.T, pr.H, pr.W, pr.heads, tiles_x, tiles_y,
                                             static_cast<int>(total), flag, gate);
    return cudaGetLastError();
}

}  // namespace

// Learned offsets below 1 in size, window (3,3,3): every corner of every sample, and the +1 neighbour a
// one-sided derivative needs when a position rounds up to a grid position, lie in the box of 6 x 6 x 6
// positions whose first corner is query - 2: the table of a (5,5,5) window.
int bounded_offsets_table_floats() { return 2 * TableShape<128, 5, 5, 5>::CELLS8; }

bool try_bounded_offsets_tables(const void* q, const void* k, const void* v, const void* dout, float* table,
                                const Problem& pr, const int* gate, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if ((pr.d != 128 && pr.d != 64) || pr.kt != 3 || pr.kh != 3 || pr.kw != 3) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    *err = pr.d == 128 ? launch_tables<128, 5, 5, 5>(q, k, v, dout, table, pr, flag, stream, &unsupported, gate)
                       : launch_tables<64, 5, 5, 5>(q, k, v, dout, table, pr, flag, stream, &unsupported, gate);
    return !unsupported;
}

// Floats per (token, head) item of the table for this problem, or 0 when the tensor-core table
// kernel does not cover it (then the backward gathers its dot products itself).
int fixed_window_table_floats(const Problem& pr, bool bf16) {
    if (!bf16 || (pr.d != 128 && pr.d != 64)) return 0;
    if (pr.kt == 3 && pr.kh == 3 && pr.kw == 3) return 2 * TableShape<128, 3, 3, 3>::CELLS8;
    if (pr.kt == 2 && pr.kh == 2 && pr.kw == 2) return 2 * TableShape<128, 2, 2, 2>::CELLS8;
    if (pr.kt == 3 && pr.kh == 5 && pr.kw == 5) return 2 * TableShape<128, 3, 5, 5>::CELLS8;
    if (pr.kt == 3 && pr.kh == 7 && pr.kw == 7) return 2 * TableShape<128, 3, 7, 7>::CELLS8;
    return 0;
}

bool try_fixed_window_tables(const void* q, const void* k, const void* v, const void* dout, float* table,
                             const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (fixed_window_table_floats(pr, true) == 0) return false;
    int* flag = timeout_flag_device_address();
    if (!flag) return false;
    bool unsupported = false;
    const bool w333 = pr.kt == 3 && pr.kh == 3, w355 = pr.kt == 3 && pr.kh == 5, w377 = pr.kt == 3 && pr.kh == 7;
    if (pr.d == 128)
        *err = w333 ? launch_tables<128, 3, 3, 3>(q, k, v, dout, table, pr, flag, stream, &unsupported)
             : w355 ? launch_tables<128, 3, 5, 5>(q, k, v, dout, table, pr, flag, stream, &unsupported)
             : w377 ? launch_tables<128, 3, 7, 7>(q, k, v, dout, table, pr, flag, stream, &unsupported)
                    : launch_tables<128, 2, 2, 2>(q, k, v, dout, table, pr, flag, stream, &unsupported);
    else
        *err = w333 ? launch_tables<64, 3, 3, 3>(q, k, v, dout, table, pr, flag, stream, &unsupported)
             : w355 ? launch_tables<64, 3, 5, 5>(q, k, v, dout, table, pr, flag, stream, &unsupported)
             : w377 ? launch_tables<64, 3, 7, 7>(q, k, v, dout, table, pr, flag, stream, &unsupported)
                    : launch_tables<64, 2, 2, 2>(q, k, v, dout, table, pr, flag, stream, &unsupported);
    return !unsupported;
}

}  // namespace dsa3d
