// dK and dV of the backward on the tensor cores, one block of keys at a time (bf16 storage, 64 or 128
// channels per head).
//
// dK[j] = sum over (query i, sample p, corner c landing on key j) of  w_c ck_{i,p} q_i  and dV[j] likewise
// with cv and dO (the chain rule through the trilinear samples of the Formulation).  Written for a block
// of 256 keys (4 x 8 x 8 positions of one head) and the queries around it, that is
//     dK_block = A_k . Q,   dV_block = A_v . dO,
// with A[key, query] = sum of the coefficients that query sends to that key: a sparse matrix (a few per
// cent of its entries), but one whose non-zeros are found without sorting anything, and whose product is
// a dense contraction the tensor cores take.  The block's result is complete when its queries have been
// walked, so it leaves the chip once - no per-contribution reductions into global memory.
//
// One persistent CTA per SM walks its blocks; for a block it walks the chunks of the block's query region
// (32 queries: 4 rows x 8 columns of one frame; 16 x 5 x 3 chunk slots, those outside the grid or the
// launch's frames skipped).  Roles:
//   two groups of four warps take the chunks alternately, each with its own pair of A matrices.  For a chunk
//     a group scans the cell codes the gather kernel left for the chunk's (query, sample) pairs and lists the
//     samples with a corner inside the block (about 6 % of them); requests their offsets and coefficient
//     pairs; once the MMAs of its previous chunk are done, puts that chunk's entries of A back to zero from
//     its list (nothing dense is swept per chunk); then adds each listed sample's up to eight coefficients
//     into A (fp32 words in shared memory, 128-byte-swizzled K-major rows of 32 queries, shared-memory
//     atomics) and hands the chunk over;
//   four warps stage the chunks' q and dO rows, widened to fp32 and transposed, as the K-major B operands
//     (one row per channel, 32 queries along it), one chunk ahead in registers;
//   one thread issues, per chunk, 16 tcgen05.mma.kind::tf32 (M = 128 keys, N = channels, K = 8 queries) that
//     accumulate into the block's four fp32 tiles in TMEM (dK and dV, two row halves).
// The tensor core reads the top 19 bits of each word: q and dO are exact (bf16), the coefficients lose the
// bits below 2^-10 relative.  When a block is done, the group that owns the next chunk adds the tiles from
// TMEM to the fp32 accumulators.
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the library's timeout flag and the
// CTA walks through the rest of its work without waiting.
#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"
#include "dsa3d_tcgen05.cuh"

namespace dsa3d {
namespace {

constexpr int kBkRows = kKbT * kKbY * kKbX;                            // 256 keys: two MMA row halves
constexpr int kBkChunkY = 4, kBkChunkX = 8, kBkChunkQ = kBkChunkY * kBkChunkX;
constexpr int kBkChunksX = kKbRegX / kBkChunkX;                        // 3
constexpr int kBkChunksPerFrame = (kKbRegY / kBkChunkY) * kBkChunksX;  // 15
constexpr int kBkSlots = kKbRegT * kBkChunksPerFrame;                  // 240 chunk slots per block
constexpr int kBkGroup = 128;                                          // threads of a scatter group
constexpr int kBkStagers = 128;                                        // threads staging the B operands
constexpr int kBkThreads = 2 * kBkGroup + kBkStagers + 32;             // + the warp that issues the MMAs
constexpr int kBkListCap = 1024;                                       // listed samples per chunk and pass (32 queries x 32 samples)
constexpr int kBkHeld = 2;                                             // listed samples a thread holds in registers
static_assert(kBkRows == 256 && kBkChunkQ == 32, "the index arithmetic below assumes these");

template <int D>
struct __align__(1024) BkSmem {
    float a32[2][2][kBkRows * kBkChunkQ];      // [group][dK, dV]: rows of 32 queries (128 bytes), 128-byte swizzle
    float b32[2][2][kBkChunkQ * D];            // [group][q, dO]: rows = channels, 32 queries (128 bytes) each, same swizzle
    uint32_t list[2][2][kBkListCap];           // [group][chunk parity]: ql | p << 5 | (rt+1) << 13 | (ry+1) << 16 | (rx+1) << 20
    uint32_t count[2][4];                      // [group][chunk % 3]
    uint32_t blk_data[2];                      // [block parity]: an MMA has written the block's tiles
    int last_seq[2];                           // [group]: block of the group's last chunk
    uint64_t bar_a_full[2], bar_b_full[2], bar_done[2];
    uint32_t tmem_base;
    uint32_t abort;
};

// What is the same for every chunk of a launch.
struct BkWalk {
    int my_blocks;                  // key blocks of this CTA
    int blocks_per_head, by_count, bx_count, tb_begin;
    int f0, f1;                     // query frames of this launch
};

struct BkChunk {
    int seq, slot;                  // which of the CTA's blocks, which chunk slot of it
    int m, t0, y0, x0;              // head and origin of the key block
    int qt, qy0, qx0;               // frame and origin of the chunk's queries
    bool valid;
};

__device__ __forceinline__ void bk_start(BkChunk& ch) {
    ch.seq = -1; ch.slot = kBkSlots; ch.m = ch.t0 = ch.y0 = ch.x0 = ch.qt = ch.qy0 = ch.qx0 = 0; ch.valid = true;
}

// Head and origin of the CTA's block number `seq`.
__device__ __forceinline__ void bk_locate(int seq, const BkWalk& wk, int& m, int& t0, int& y0, int& x0) {
    const int item = static_cast<int>(blockIdx.x) + seq * static_cast<int>(gridDim.x);
    m = item / wk.blocks_per_head;
    int rem = item - m * wk.blocks_per_head;
    x0 = (rem % wk.bx_count) * kKbX; rem /= wk.bx_count;
    y0 = (rem % wk.by_count) * kKbY;
    t0 = (wk.tb_begin + rem / wk.by_count) * kKbT;
}

// Next chunk slot that holds queries of this launch (every role of the CTA walks the same sequence).
__device__ __forceinline__ void bk_advance(BkChunk& ch, const BkWalk& wk, const Problem& pr) {
    if (!ch.valid) return;
    for (;;) {
        if (++ch.slot >= kBkSlots) {
            if (++ch.seq >= wk.my_blocks) { ch.valid = false; return; }
            bk_locate(ch.seq, wk, ch.m, ch.t0, ch.y0, ch.x0);
            ch.slot = 0;
        }
        const int frame = ch.slot / kBkChunksPerFrame;
        ch.qt = ch.t0 - kKbLoT + frame;
        if (ch.qt < wk.f0) { ch.slot = (wk.f0 - (ch.t0 - kKbLoT)) * kBkChunksPerFrame - 1; continue; }
        if (ch.qt >= wk.f1) { ch.slot = kBkSlots; continue; }
        const int r = ch.slot - frame * kBkChunksPerFrame;
        ch.qy0 = ch.y0 - kKbLoY + kBkChunkY * (r / kBkChunksX);
        ch.qx0 = ch.x0 - kKbLoX + kBkChunkX * (r % kBkChunksX);
        if (ch.qy0 + kBkChunkY <= 0 || ch.qy0 >= pr.H || ch.qx0 + kBkChunkX <= 0 || ch.qx0 >= pr.W) continue;
        return;
    }
}

__device__ __forceinline__ void bk_named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Element (key row, query) of an A matrix: rows of 32 fp32, the 16-byte pieces of a row exchanged by the
// 128-byte swizzle.
__device__ __forceinline__ int bk_a_index(int row, int ql) {
    return row * kBkChunkQ + ((((ql >> 2) ^ (row & 7)) << 2) | (ql & 3));
}

template <int D, bool MULTI>      // MULTI: more than 32 samples per query, taken in passes of 32
__global__ void __launch_bounds__(kBkThreads, 1)
dkdv_block_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ dout,
                  const float* __restrict__ offsets, const float2* __restrict__ coef, float* __restrict__ acc_dk,
                  float* __restrict__ acc_dv, const int total_blocks, const int blocks_per_head, const int by_count,
                  const int bx_count, const int tb_begin, const int f0, const int f1, int* timeout_flag,
                  const Problem pr) {
    extern __shared__ unsigned char raw[];
    BkSmem<D>& s = *reinterpret_cast<BkSmem<D>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kMmaWarp = (2 * kBkGroup + kBkStagers) / 32;
    const uint32_t* __restrict__ codes_g = pr.cell_codes;
    [[maybe_unused]] const long long code_extent = pr.N * pr.heads * pr.P;
    [[maybe_unused]] const long long kv_extent = pr.N * pr.heads * D;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s.bar_a_full[i]), kBkGroup / 32);      // lane 0 of every warp of the group
            mbar_init(smem_u32(&s.bar_b_full[i]), kBkStagers / 32);
            mbar_init(smem_u32(&s.bar_done[i]), 1);
            for (int k = 0; k < 4; ++k) s.count[i][k] = 0u;
            s.blk_data[i] = 0u;
            s.last_seq[i] = -1;
        }
        s.abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s.tmem_base)), "r"(4 * D));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    {   // the A matrices start as zeros and are put back to zeros after each use
        float4* a = reinterpret_cast<float4*>(&s.a32[0][0][0]);
        for (int i = tid; i < 2 * 2 * kBkRows * kBkChunkQ / 4; i += kBkThreads) a[i] = make_float4(0.f, 0.f, 0.f, 0.f);
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

    BkWalk wk;
    wk.my_blocks = static_cast<int>(blockIdx.x) < total_blocks
                       ? (total_blocks - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x) : 0;
    wk.blocks_per_head = blocks_per_head; wk.by_count = by_count; wk.bx_count = bx_count; wk.tb_begin = tb_begin;
    wk.f0 = f0; wk.f1 = f1;

    if (warp == kMmaWarp) {
        // ==================================================================== MMA thread
        if (lane == 0) {
            // D fp32, A and B tf32, both K-major (an MN-major tf32 operand was measured to yield zeros), N = D, M = 128
            constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (static_cast<uint32_t>(D >> 3) << 17) |
                                       (static_cast<uint32_t>(128 >> 4) << 24);
            uint64_t desc_a[2][2], desc_b[2][2];
            for (int g = 0; g < 2; ++g)
                for (int x = 0; x < 2; ++x) {
                    desc_a[g][x] = smem_desc(smem_u32(&s.a32[g][x][0]));
                    desc_b[g][x] = smem_desc(smem_u32(&s.b32[g][x][0]));
                }
            BkChunk ch;
            bk_start(ch);
            bk_advance(ch, wk, pr);
            int cur = -1;
            bool fresh = true;
            for (int j = 0; ch.valid; ++j) {
                const int g = j & 1, i = j >> 1;
                if (ch.seq != cur) { cur = ch.seq; fresh = true; }
                bool ok = wait(&s.bar_a_full[g], static_cast<uint32_t>(i & 1), 31);
                if (ok) ok = wait(&s.bar_b_full[g], static_cast<uint32_t>(i & 1), 35);
                if (ok) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (*(volatile uint32_t*)&s.count[g][i % 3] > 0u) {
                        if (fresh) { *(volatile uint32_t*)&s.blk_data[cur & 1] = 1u; __threadfence_block(); }
#pragma unroll
                        for (int x = 0; x < 2; ++x)
#pragma unroll
                            for (int half = 0; half < 2; ++half)
#pragma unroll
                                for (int ks = 0; ks < 4; ++ks)
                                    umma_tf32(tmem + static_cast<uint32_t>((2 * x + half) * D),
                                              desc_a[g][x] + static_cast<uint64_t>(half * (128 * 128 >> 4) + 2 * ks),
                                              desc_b[g][x] + static_cast<uint64_t>(2 * ks), idesc, (ks > 0 || !fresh) ? 1u : 0u);
                        fresh = false;
                    }
                }
                umma_commit(smem_u32(&s.bar_done[g]));                // arrives at once if nothing was issued
                bk_advance(ch, wk, pr);
            }
        }
    } else if (warp >= 2 * kBkGroup / 32) {
        // ==================================================================== B operands: lane = query, warp = channel range
        constexpr int CPS = D / (kBkStagers / 32);                    // channels per warp
        constexpr int UPS = CPS / 8;                                  // 16-byte pieces of them
        const int sw = warp - 2 * kBkGroup / 32;
        uint4 rows_q[UPS], rows_d[UPS];
        auto load_rows = [&](const BkChunk& ch) {
            const int qy = ch.qy0 + (lane >> 3), qx = ch.qx0 + (lane & 7);
            const bool in_grid = ch.valid && qy >= 0 && qy < pr.H && qx >= 0 && qx < pr.W;
            const long long o_ = (((static_cast<long long>(ch.qt) * pr.H + qy) * pr.W + qx) * pr.heads + ch.m) * D + sw * CPS;
#pragma unroll
            for (int u = 0; u < UPS; ++u) {
                rows_q[u] = rows_d[u] = make_uint4(0u, 0u, 0u, 0u);
                if (in_grid && DSA3D_IN_RANGE(pr, o_ + u * 8, kv_extent, 15)) {
                    rows_q[u] = __ldg(reinterpret_cast<const uint4*>(q + o_) + u);
                    rows_d[u] = __ldg(reinterpret_cast<const uint4*>(dout + o_) + u);
                }
            }
        };
        BkChunk ch;
        bk_start(ch);
        bk_advance(ch, wk, pr);
        load_rows(ch);
        for (int j = 0; ch.valid; ++j) {
            const int g = j & 1, i = j >> 1;
            if (i >= 1) wait(&s.bar_done[g], static_cast<uint32_t>((i - 1) & 1), 36);     // the MMAs of chunk j - 2 have read this buffer
            float* bq = &s.b32[g][0][0];
            float* bd = &s.b32[g][1][0];
#pragma unroll
            for (int u = 0; u < UPS; ++u) {
                const uint32_t wq[4] = {rows_q[u].x, rows_q[u].y, rows_q[u].z, rows_q[u].w};
                const uint32_t wd[4] = {rows_d[u].x, rows_d[u].y, rows_d[u].z, rows_d[u].w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int n = sw * CPS + u * 8 + e;
                    const int at = n * kBkChunkQ + ((((lane >> 2) ^ (n & 7)) << 2) | (lane & 3));
                    bq[at] = __uint_as_float((e & 1) ? (wq[e >> 1] & 0xffff0000u) : (wq[e >> 1] << 16));
                    bd[at] = __uint_as_float((e & 1) ? (wd[e >> 1] & 0xffff0000u) : (wd[e >> 1] << 16));
                }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_b_full[g]));
            bk_advance(ch, wk, pr);
            load_rows(ch);
        }
    } else {
        // ==================================================================== scatter groups
        const int g = warp / (kBkGroup / 32), gt = tid - g * kBkGroup, gw = gt >> 5;
        const int bar_id = 1 + g;
        float* a_k = &s.a32[g][0][0];
        float* a_v = &s.a32[g][1][0];
        volatile uint32_t* counts = s.count[g];
        // a listed sample: its offsets and coefficient pair, then its coefficients into the A matrices
        auto load_details = [&](uint32_t entry, const BkChunk& ch, float (&o)[3], float2& cf) {
            const int ql = entry & 31, p = (entry >> 5) & 255;
            const long long n = (static_cast<long long>(ch.qt) * pr.H + (ch.qy0 + (ql >> 3))) * pr.W + (ch.qx0 + (ql & 7));
            const long long sample = (n * pr.heads + ch.m) * pr.P + p;
            o[0] = o[1] = o[2] = 0.0f; cf = make_float2(0.f, 0.f);
            if (DSA3D_IN_RANGE(pr, sample, code_extent, 11)) {
                o[0] = __ldg(offsets + sample * 3); o[1] = __ldg(offsets + sample * 3 + 1); o[2] = __ldg(offsets + sample * 3 + 2);
                cf = __ldg(coef + sample);
            }
        };
        auto scatter = [&](uint32_t entry, const BkChunk& ch, const float (&o)[3], const float2 cf) {
            const int ql = entry & 31, p = (entry >> 5) & 255;
            const Cell cell = make_cell_values(pr, ch.qt, ch.qy0 + (ql >> 3), ch.qx0 + (ql & 7), p, o[0], o[1], o[2]);
            const int rt = cell.it - ch.t0, ry = cell.iy - ch.y0, rx = cell.ix - ch.x0;
            const float wt[2] = {1.0f - cell.ft, cell.ft}, wy[2] = {1.0f - cell.fy, cell.fy}, wx[2] = {1.0f - cell.fx, cell.fx};
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int kt_ = rt + (c >> 2), ky_ = ry + ((c >> 1) & 1), kx_ = rx + (c & 1);
                const float w = wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1];
                if (((cell.mask >> c) & 1u) && w != 0.0f && static_cast<unsigned>(kt_) < static_cast<unsigned>(kKbT) &&
                    static_cast<unsigned>(ky_) < static_cast<unsigned>(kKbY) && static_cast<unsigned>(kx_) < static_cast<unsigned>(kKbX)) {
                    const int idx = bk_a_index((kt_ * kKbY + ky_) * kKbX + kx_, ql);
                    atomicAdd(a_k + idx, w * cf.x);
                    atomicAdd(a_v + idx, w * cf.y);
                }
            }
        };
        // the entries of A that the samples of a list may have touched, back to zero
        auto clear_listed = [&](const uint32_t* lst, int n) {
            for (int pair = gt; pair < n * 8; pair += kBkGroup) {
                const uint32_t entry = lst[pair >> 3];
                const int cc = pair & 7;
                const int kt_ = static_cast<int>((entry >> 13) & 7u) - 1 + (cc >> 2);
                const int ky_ = static_cast<int>((entry >> 16) & 15u) - 1 + ((cc >> 1) & 1);
                const int kx_ = static_cast<int>((entry >> 20) & 15u) - 1 + (cc & 1);
                if (static_cast<unsigned>(kt_) < static_cast<unsigned>(kKbT) && static_cast<unsigned>(ky_) < static_cast<unsigned>(kKbY) &&
                    static_cast<unsigned>(kx_) < static_cast<unsigned>(kKbX)) {
                    const int idx = bk_a_index((kt_ * kKbY + ky_) * kKbX + kx_, static_cast<int>(entry & 31u));
                    a_k[idx] = 0.0f;
                    a_v[idx] = 0.0f;
                }
            }
        };
        // samples of the group's 32 queries x 32 lanes whose cell touches the block -> list
        auto scan = [&](const uint32_t (&codes)[8], int pi, const BkChunk& ch, uint32_t* lst, uint32_t* counter) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t code = codes[k];
                const uint32_t dt = (code & 1023u) - static_cast<uint32_t>(ch.t0);          // corner 0 relative to the block, + 1
                const uint32_t dy = ((code >> 10) & 1023u) - static_cast<uint32_t>(ch.y0);
                const uint32_t dx = (code >> 20) - static_cast<uint32_t>(ch.x0);
                if (code != kDeadCellCode && dt <= static_cast<uint32_t>(kKbT) && dy <= static_cast<uint32_t>(kKbY) &&
                    dx <= static_cast<uint32_t>(kKbX)) {
                    const uint32_t at = atomicAdd(counter, 1u);
                    if (at < static_cast<uint32_t>(kBkListCap))
                        lst[at] = static_cast<uint32_t>(gw * 8 + k) | (static_cast<uint32_t>(pi * 32 + lane) << 5) | (dt << 13) | (dy << 16) | (dx << 20);
                }
            }
        };
        auto load_codes = [&](uint32_t (&codes)[8], int pi, const BkChunk& ch) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int ql = gw * 8 + k;
                const int qy = ch.qy0 + (ql >> 3), qx = ch.qx0 + (ql & 7), p = pi * 32 + lane;
                const long long at = ((((static_cast<long long>(ch.qt) * pr.H + qy) * pr.W + qx) * pr.heads + ch.m)) * pr.P + p;
                codes[k] = kDeadCellCode;
                if (ch.valid && qy >= 0 && qy < pr.H && qx >= 0 && qx < pr.W && p < pr.P && DSA3D_IN_RANGE(pr, at, code_extent, 14))
                    codes[k] = __ldg(codes_g + at);
            }
        };
        // the finished block: its four tiles from TMEM to the accumulators (warp of the group = TMEM lane quarter)
        auto epilogue = [&](int seq) {
            int m, t0, y0, x0;
            bk_locate(seq, wk, m, t0, y0, x0);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
            for (int tile = 0; tile < 4; ++tile) {
                const int x = tile >> 1, half = tile & 1;
                float* acc = x ? acc_dv : acc_dk;
                const int r = half * 128 + gw * 32 + lane;
                const int kt_ = t0 + r / (kKbY * kKbX), ky_ = y0 + (r / kKbX) % kKbY, kx_ = x0 + r % kKbX;
                const bool in_grid = kt_ < pr.T && ky_ < pr.H && kx_ < pr.W;
                const long long o_ = (((static_cast<long long>(kt_) * pr.H + ky_) * pr.W + kx_) * pr.heads + m) * D;
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t regs[32];
                    tmem_load_32(tmem + (static_cast<uint32_t>(gw * 32) << 16) + static_cast<uint32_t>(tile * D + c0), regs);
                    if (in_grid && !*abort_flag && DSA3D_IN_RANGE(pr, o_, kv_extent, 13)) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            red_add_v4(acc + o_ + c0 + e, __uint_as_float(regs[e]), __uint_as_float(regs[e + 1]),
                                       __uint_as_float(regs[e + 2]), __uint_as_float(regs[e + 3]));
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        };

        BkChunk ch;
        bk_start(ch);
        bk_advance(ch, wk, pr);
        int j = 0, prev_seq = -1, last_seq = -1;
        if (g == 1) {
            if (ch.valid) prev_seq = ch.seq;
            bk_advance(ch, wk, pr);
            j = 1;
        }
        uint32_t codes[8];
        if constexpr (!MULTI) load_codes(codes, 0, ch);
        for (int i = 0; ch.valid; ++i, j += 2) {
            BkChunk nx = ch;
            bk_advance(nx, wk, pr);
            const int mid_seq = nx.valid ? nx.seq : -1;                  // block of the chunk between this one and the group's next
            bk_advance(nx, wk, pr);
            uint32_t* lst = s.list[g][i & 1];
            uint32_t* counter = &s.count[g][i % 3];
            bool drained = false;
            if constexpr (!MULTI) {
                // ---- which samples touch the block; their details requested; the codes of the group's next chunk requested
                scan(codes, 0, ch, lst, counter);
                bk_named_barrier(bar_id, kBkGroup);
                const int n = static_cast<int>(min(counts[i % 3], static_cast<uint32_t>(kBkListCap)));
                uint32_t ent[kBkHeld];
                float o[kBkHeld][3];
                float2 cf[kBkHeld];
#pragma unroll
                for (int h = 0; h < kBkHeld; ++h) {
                    ent[h] = 0u;
                    if (gt + h * kBkGroup < n) { ent[h] = lst[gt + h * kBkGroup]; load_details(ent[h], ch, o[h], cf[h]); }
                }
                load_codes(codes, 0, nx);
                if (gt == 0) s.count[g][(i + 1) % 3] = 0u;               // the count of chunk i - 2 is no longer read
                // ---- the previous chunk has been multiplied: its entries of A back to zero (and a finished block out)
                if (i >= 1) wait(&s.bar_done[g], static_cast<uint32_t>((i - 1) & 1), 33);
                if (j > 0 && ch.seq != prev_seq) {
                    wait(&s.bar_done[g ^ 1], static_cast<uint32_t>(((j - 1) >> 1) & 1), 32);
                    if (*(volatile uint32_t*)&s.blk_data[prev_seq & 1]) { epilogue(prev_seq); drained = true; }
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (i >= 1) clear_listed(s.list[g][(i - 1) & 1], static_cast<int>(min(counts[(i - 1) % 3], static_cast<uint32_t>(kBkListCap))));
                bk_named_barrier(bar_id, kBkGroup);
                if (drained && gt == 0) *(volatile uint32_t*)&s.blk_data[prev_seq & 1] = 0u;
                // ---- this chunk's coefficients into A
#pragma unroll
                for (int h = 0; h < kBkHeld; ++h)
                    if (gt + h * kBkGroup < n) scatter(ent[h], ch, o[h], cf[h]);
                for (int base = kBkHeld * kBkGroup; base < n; base += kBkHeld * kBkGroup) {
#pragma unroll
                    for (int h = 0; h < kBkHeld; ++h) {
                        ent[h] = 0u;
                        if (base + gt + h * kBkGroup < n) { ent[h] = lst[base + gt + h * kBkGroup]; load_details(ent[h], ch, o[h], cf[h]); }
                    }
#pragma unroll
                    for (int h = 0; h < kBkHeld; ++h)
                        if (base + gt + h * kBkGroup < n) scatter(ent[h], ch, o[h], cf[h]);
                }
            } else {
                // ---- more than 32 samples per query: the previous chunk's A cleared whole, then one pass per 32 samples
                if (gt == 0) { s.count[g][(i + 1) % 3] = 0u; }
                if (i >= 1) wait(&s.bar_done[g], static_cast<uint32_t>((i - 1) & 1), 33);
                if (j > 0 && ch.seq != prev_seq) {
                    wait(&s.bar_done[g ^ 1], static_cast<uint32_t>(((j - 1) >> 1) & 1), 32);
                    if (*(volatile uint32_t*)&s.blk_data[prev_seq & 1]) { epilogue(prev_seq); drained = true; }
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (i >= 1) {
                    float4* a = reinterpret_cast<float4*>(a_k);              // dK and dV matrices are adjacent
                    for (int e = gt; e < 2 * kBkRows * kBkChunkQ / 4; e += kBkGroup) a[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                uint32_t* pass_counter = &s.count[g][3];
                const int passes = (pr.P + 31) / 32;
                for (int pi = 0; pi < passes; ++pi) {
                    if (gt == 0) *pass_counter = 0u;
                    load_codes(codes, pi, ch);
                    bk_named_barrier(bar_id, kBkGroup);
                    if (drained && gt == 0 && pi == 0) *(volatile uint32_t*)&s.blk_data[prev_seq & 1] = 0u;
                    scan(codes, pi, ch, lst, pass_counter);
                    bk_named_barrier(bar_id, kBkGroup);
                    const int n = static_cast<int>(min(counts[3], static_cast<uint32_t>(kBkListCap)));
                    if (gt == 0) *counter += static_cast<uint32_t>(n);
                    for (int base = 0; base < n; base += kBkHeld * kBkGroup) {
                        uint32_t ent[kBkHeld];
                        float o[kBkHeld][3];
                        float2 cf[kBkHeld];
#pragma unroll
                        for (int h = 0; h < kBkHeld; ++h) {
                            ent[h] = 0u;
                            if (base + gt + h * kBkGroup < n) { ent[h] = lst[base + gt + h * kBkGroup]; load_details(ent[h], ch, o[h], cf[h]); }
                        }
#pragma unroll
                        for (int h = 0; h < kBkHeld; ++h)
                            if (base + gt + h * kBkGroup < n) scatter(ent[h], ch, o[h], cf[h]);
                    }
                    bk_named_barrier(bar_id, kBkGroup);
                }
            }
            fence_async_smem();                                       // the MMAs read A through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_a_full[g]));
            last_seq = ch.seq;
            prev_seq = mid_seq;
            ch = nx;
        }
        // ---- the last block: every MMA done, then group 0 takes it out
        {
            const int i_last = (j - 2 - g) / 2;                       // the group's last chunk (j has moved one step past it)
            if (last_seq >= 0) wait(&s.bar_done[g], static_cast<uint32_t>(i_last & 1), 34);
            if (gt == 0) s.last_seq[g] = last_seq;
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            bk_named_barrier(3, 2 * kBkGroup);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (g == 0) {
                const int a = *(volatile int*)&s.last_seq[0], b = *(volatile int*)&s.last_seq[1];
                const int seq = a > b ? a : b;
                if (seq >= 0 && *(volatile uint32_t*)&s.blk_data[seq & 1]) epilogue(seq);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kMmaWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(4 * D));
}

template <int D, bool MULTI>
cudaError_t launch_blocks_t(const void* q, const void* dout, const float* offsets, const float2* coef, float* acc_dk,
                            float* acc_dv, int total, int per_head, int by_count, int bx_count, int tb_begin, int f0, int f1,
                            int* flag, const Problem& pr, cudaStream_t stream) {
    auto kern = dkdv_block_kernel<D, MULTI>;
    const size_t smem = sizeof(BkSmem<D>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kBkThreads, smem, stream>>>(static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(dout),
                                             offsets, coef, acc_dk, acc_dv, total, per_head, by_count, bx_count, tb_begin,
                                             f0, f1, flag, pr);
    return cudaGetLastError();
}

}  // namespace

bool key_blocks_shape_covered(const Problem& pr) {
    if (pr.d != 128 && pr.d != 64) return false;
    if (pr.T > 1022 || pr.H > 1022 || pr.W > 1022 || pr.P > 256) return false;       // 10-bit fields of the cell codes
    const long long blocks = static_cast<long long>((pr.T + kKbT - 1) / kKbT) * ((pr.H + kKbY - 1) / kKbY) *
                             ((pr.W + kKbX - 1) / kKbX) * pr.heads;
    return blocks < (1LL << 30);
}

cudaError_t launch_dkdv_blocks(const void* q, const void* dout, const float* offsets, const float2* coef, float* acc_dk,
                               float* acc_dv, const Problem& pr, cudaStream_t stream) {
    if (!key_blocks_shape_covered(pr) || !pr.cell_codes) return cudaErrorInvalidValue;
    int* flag = timeout_flag_device_address();
    if (!flag) return cudaErrorInvalidValue;
    const long long per_frame = static_cast<long long>(pr.H) * pr.W;
    const int f0 = static_cast<int>(pr.q_begin / per_frame), f1 = static_cast<int>((pr.q_begin + pr.q_count) / per_frame);
    if (f1 <= f0) return cudaSuccess;
    // key blocks whose region [t0 - 6, t0 + 10) meets the frames [f0, f1)
    const int lo = f0 - (kKbRegT - kKbLoT) + 1;
    const int tb_begin = lo <= 0 ? 0 : (lo + kKbT - 1) / kKbT;
    int tb_end = (f1 + kKbLoT - 1) / kKbT;                                         // last block with t0 - 6 < f1
    if (tb_end > (pr.T - 1) / kKbT) tb_end = (pr.T - 1) / kKbT;
    if (tb_end < tb_begin) return cudaSuccess;
    const int by_count = (pr.H + kKbY - 1) / kKbY, bx_count = (pr.W + kKbX - 1) / kKbX;
    const int per_head = (tb_end - tb_begin + 1) * by_count * bx_count;
    const int total = per_head * pr.heads;
#define DSA3D_BK(DD, MM) launch_blocks_t<DD, MM>(q, dout, offsets, coef, acc_dk, acc_dv, total, per_head, by_count, bx_count, \
                                                 tb_begin, f0, f1, flag, pr, stream)
    if (pr.d == 128) return pr.P <= 32 ? DSA3D_BK(128, false) : DSA3D_BK(128, true);
    return pr.P <= 32 ? DSA3D_BK(64, false) : DSA3D_BK(64, true);
#undef DSA3D_BK
}

}  // namespace dsa3d
