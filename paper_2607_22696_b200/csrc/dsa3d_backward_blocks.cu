// dK and dV of the backward on the tensor cores, one block of keys at a time (bf16 storage, 64 or 128
// channels per head).
//
// dK[j] = sum over (query i, sample p, corner c landing on key j) of  w_c ck_{i,p} q_i  and dV[j] likewise
// with cv and dO (the chain rule through the trilinear samples of the Formulation).  Written for a block
// of 256 keys (4 x 8 x 8 positions of one head) and the queries around it, that is
//     dK_block = A_k . Q,   dV_block = A_v . dO,
// with A[key, query] = sum of the coefficients that query sends to that key: a sparse matrix (a few per
// cent of its entries) whose product is a dense contraction the tensor cores take.  The block's result is
// complete when its queries have been walked, so it leaves the chip once.
//
// The gather kernel has appended every sample to the list of each key block it touches
// (block_lists_append).  One persistent CTA per SM walks its blocks; for a block it walks the chunks of
// the block's query region (32 queries: 4 rows x 8 columns of one frame; 16 x 5 x 3 chunk slots, those
// outside the grid or the launch's frames skipped).  Roles:
//   four sorter warps, one block ahead: a counting sort of the block's list by chunk slot, during which they
//     fetch each sample's offsets and coefficient pair, form its cell once more (make_cell_values: the same
//     arithmetic as the gather kernel) and write, for every corner of the sample that lies in the block, a
//     16-byte entry {position in A, w_c ck, w_c cv} to the CTA's scratch in global memory, chunk after chunk;
//   two groups of four warps take the chunks alternately, each with its own pair of A matrices (fp32 words,
//     128-byte-swizzled K-major rows of 32 queries): once the MMAs of the group's previous chunk are done its
//     entries of A go back to zero from a list of positions in shared memory (nothing dense is swept per
//     chunk), then the chunk's entries - already on their way into registers - are added with shared-memory
//     atomics and the chunk is handed over;
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
constexpr int kBkChunkY = kKbChunkY, kBkChunkX = kKbChunkX, kBkChunkQ = kBkChunkY * kBkChunkX;
constexpr int kBkChunksX = kKbChunksX;                                 // 3
constexpr int kBkChunksPerFrame = kKbChunksPerFrame;                   // 15
constexpr int kBkSlots = kKbRegT * kBkChunksPerFrame;                  // 240 chunk slots per block
constexpr int kBkGroup = 128;                                          // threads of a scatter group
constexpr int kBkStagers = 128;                                        // threads staging the B operands
constexpr int kBkSorters = 128;                                        // threads sorting the next block's list
constexpr int kBkThreads = 2 * kBkGroup + kBkStagers + kBkSorters + 32;   // + the warp that issues the MMAs
constexpr int kBkListCap = 2048;                                       // positions of a chunk remembered for the sparse clear
constexpr int kBkHeld = 4;                                             // entries a thread holds in registers
constexpr int kBkMaxCtas = 160;                                        // resident CTAs the sorted scratch is sized for
static_assert(kBkRows == 256 && kBkChunkQ == 32 && kBkSlots <= 256, "the index arithmetic below assumes these");

using BkEntry = uint4;                     // {position in A (bk_a_index), fp32 w*ck, fp32 w*cv, unused}

template <int D>
struct __align__(1024) BkSmem {
    float a32[2][2][kBkRows * kBkChunkQ];      // [group][dK, dV]: rows of 32 queries (128 bytes), 128-byte swizzle
    float b32[2][2][kBkChunkQ * D];            // [group][q, dO]: rows = channels, 32 queries (128 bytes) each, same swizzle
    uint16_t list[2][2][kBkListCap];           // [group][chunk parity]: positions the chunk touched, for the clear
    uint32_t chunk_start[2][kBkSlots + 1];     // [block parity]: first entry of every chunk slot
    uint32_t cursor[kBkSlots];                 // the sorters' histogram, then their write positions
    uint32_t count[2][2];                      // [group][chunk parity]: entries of the chunk
    uint32_t blk_data[2];                      // [block parity]: an MMA has written the block's tiles
    int last_seq[2];                           // [group]: block of the group's last chunk
    uint64_t bar_a_full[2], bar_b_full[2], bar_done[2], bar_sorted[2], bar_free[2];
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
    int frame, yc, xc;              // the slot as (frame of the region, strip of rows, strip of columns)
    int m, t0, y0, x0;              // head and origin of the key block
    int qt, qy0, qx0;               // frame and origin of the chunk's queries
    bool valid;
};

__device__ __forceinline__ void bk_start(BkChunk& ch) {
    ch.seq = -1; ch.slot = kBkSlots; ch.frame = ch.yc = ch.xc = 0;
    ch.m = ch.t0 = ch.y0 = ch.x0 = ch.qt = ch.qy0 = ch.qx0 = 0; ch.valid = true;
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
        if (ch.slot >= kBkSlots - 1) {
            if (++ch.seq >= wk.my_blocks) { ch.valid = false; return; }
            bk_locate(ch.seq, wk, ch.m, ch.t0, ch.y0, ch.x0);
            ch.slot = 0; ch.frame = ch.yc = ch.xc = 0;
        } else {
            ++ch.slot;
            if (++ch.xc == kBkChunksX) { ch.xc = 0; if (++ch.yc == kKbRegY / kBkChunkY) { ch.yc = 0; ++ch.frame; } }
        }
        ch.qt = ch.t0 - kKbLoT + ch.frame;
        if (ch.qt < wk.f0) {                                          // on to the first frame of the launch
            ch.frame = wk.f0 - (ch.t0 - kKbLoT);
            if (ch.frame >= kKbRegT) { ch.slot = kBkSlots - 1; continue; }
            ch.yc = ch.xc = 0; ch.slot = ch.frame * kBkChunksPerFrame; ch.qt = wk.f0;
        }
        if (ch.qt >= wk.f1) { ch.slot = kBkSlots - 1; continue; }
        ch.qy0 = ch.y0 - kKbLoY + kBkChunkY * ch.yc;
        ch.qx0 = ch.x0 - kKbLoX + kBkChunkX * ch.xc;
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

template <int D>
__global__ void __launch_bounds__(kBkThreads, 1)
dkdv_block_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ dout,
                  const float* __restrict__ offsets, const float2* __restrict__ coef, float* __restrict__ acc_dk,
                  float* __restrict__ acc_dv, BkEntry* __restrict__ sorted, const int total_blocks,
                  const int blocks_per_head, const int by_count, const int bx_count, const int tb_begin, const int f0,
                  const int f1, int* timeout_flag, const Problem pr) {
    extern __shared__ unsigned char raw[];
    BkSmem<D>& s = *reinterpret_cast<BkSmem<D>*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kStagerWarp0 = 2 * kBkGroup / 32, kSorterWarp0 = kStagerWarp0 + kBkStagers / 32,
                  kMmaWarp = kSorterWarp0 + kBkSorters / 32;
    [[maybe_unused]] const long long sample_extent = pr.N * pr.heads * pr.P;
    [[maybe_unused]] const long long kv_extent = pr.N * pr.heads * D;
    // this CTA's two buffers of sorted entries
    BkEntry* const my_sorted = sorted + static_cast<long long>(blockIdx.x) * 2 * pr.blk_cap * 8;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s.bar_a_full[i]), kBkGroup / 32);      // lane 0 of every warp of the group
            mbar_init(smem_u32(&s.bar_b_full[i]), kBkStagers / 32);
            mbar_init(smem_u32(&s.bar_done[i]), 1);
            mbar_init(smem_u32(&s.bar_sorted[i]), kBkSorters / 32);
            mbar_init(smem_u32(&s.bar_free[i]), 1);
            s.count[i][0] = s.count[i][1] = 0u;
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
    const int bt_n = (pr.T + kKbT - 1) / kKbT;

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
                    if (*(volatile uint32_t*)&s.count[g][i & 1] > 0u) {
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
    } else if (warp >= kSorterWarp0) {
        // ==================================================================== sorters: one block ahead of the groups
        const int st = tid - kSorterWarp0 * 32;
        for (int seq = 0; seq < wk.my_blocks; ++seq) {
            const int buf = seq & 1;
            // the groups have left block seq - 2, whose records and chunk starts this block replaces
            if (seq >= 2) wait(&s.bar_free[buf], static_cast<uint32_t>(((seq >> 1) - 1) & 1), 37);
            int m, t0, y0, x0;
            bk_locate(seq, wk, m, t0, y0, x0);
            const long long bid = ((static_cast<long long>(m) * bt_n + t0 / kKbT) * by_count + y0 / kKbY) * bx_count + x0 / kKbX;
            const int n = static_cast<int>(min(__ldcg(pr.blk_count + bid), static_cast<uint32_t>(pr.blk_cap)));
            const uint32_t* lst = pr.blk_list + bid * pr.blk_cap;
            for (int i = st; i < kBkSlots; i += kBkSorters) s.cursor[i] = 0u;
            bk_named_barrier(4, kBkSorters);
            // corners of a listed sample that lie in the block and in the grid (what it will add entries for)
            auto block_corners = [&](uint32_t entry) -> unsigned {
                const int rt = static_cast<int>((entry >> 21) & 7u) - 1, ry = static_cast<int>((entry >> 24) & 15u) - 1,
                          rx = static_cast<int>(entry >> 28) - 1;
                return corner_mask(rt, ry, rx, kKbT, kKbY, kKbX) & corner_mask(t0 + rt, y0 + ry, x0 + rx, pr.T, pr.H, pr.W);
            };
            for (int e = st; e < n; e += kBkSorters) {
                const uint32_t entry = __ldcg(lst + e);
                atomicAdd(&s.cursor[entry & 255u], static_cast<uint32_t>(__popc(block_corners(entry))));
            }
            bk_named_barrier(4, kBkSorters);
            if (st < 32) {                                             // exclusive prefix of the 240 counts
                constexpr int PER = (kBkSlots + 31) / 32;
                uint32_t c[PER], sum = 0u;
#pragma unroll
                for (int k = 0; k < PER; ++k) { c[k] = st * PER + k < kBkSlots ? s.cursor[st * PER + k] : 0u; sum += c[k]; }
                uint32_t incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o); if (st >= o) incl += v; }
                uint32_t run = incl - sum;
#pragma unroll
                for (int k = 0; k < PER; ++k)
                    if (st * PER + k < kBkSlots) { s.chunk_start[buf][st * PER + k] = run; s.cursor[st * PER + k] = run; run += c[k]; }
                if (st == 31) s.chunk_start[buf][kBkSlots] = incl;
            }
            bk_named_barrier(4, kBkSorters);
            BkEntry* out = my_sorted + static_cast<long long>(buf) * pr.blk_cap * 8;
            for (int e0 = st; e0 < n; e0 += 2 * kBkSorters) {
                uint32_t entry[2];
                float o[2][3];
                float2 cf[2];
                int qt[2], qy[2], qx[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int e = e0 + h * kBkSorters;
                    entry[h] = 0u; o[h][0] = o[h][1] = o[h][2] = 0.0f; cf[h] = make_float2(0.f, 0.f); qt[h] = qy[h] = qx[h] = 0;
                    if (e < n) {
                        entry[h] = __ldcg(lst + e);
                        const int slot = entry[h] & 255u, ql = (entry[h] >> 8) & 31u, p = (entry[h] >> 13) & 255u;
                        const int frame = slot / kBkChunksPerFrame, r = slot - frame * kBkChunksPerFrame;
                        qt[h] = t0 - kKbLoT + frame;
                        qy[h] = y0 - kKbLoY + kBkChunkY * (r / kBkChunksX) + (ql >> 3);
                        qx[h] = x0 - kKbLoX + kBkChunkX * (r % kBkChunksX) + (ql & 7);
                        const long long sample = (((static_cast<long long>(qt[h]) * pr.H + qy[h]) * pr.W + qx[h]) * pr.heads + m) * pr.P + p;
                        if (DSA3D_IN_RANGE(pr, sample, sample_extent, 11)) {
                            o[h][0] = __ldg(offsets + sample * 3); o[h][1] = __ldg(offsets + sample * 3 + 1); o[h][2] = __ldg(offsets + sample * 3 + 2);
                            cf[h] = __ldg(coef + sample);
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int e = e0 + h * kBkSorters;
                    if (e < n) {
                        const Cell cell = make_cell_values(pr, qt[h], qy[h], qx[h], (entry[h] >> 13) & 255u, o[h][0], o[h][1], o[h][2]);
                        const unsigned corners = block_corners(entry[h]);
                        const int ql = (entry[h] >> 8) & 31u;
                        const int rt = static_cast<int>((entry[h] >> 21) & 7u) - 1, ry = static_cast<int>((entry[h] >> 24) & 15u) - 1,
                                  rx = static_cast<int>(entry[h] >> 28) - 1;
                        uint32_t at = atomicAdd(&s.cursor[entry[h] & 255u], static_cast<uint32_t>(__popc(corners)));
                        const float wt[2] = {1.0f - cell.ft, cell.ft}, wy[2] = {1.0f - cell.fy, cell.fy}, wx[2] = {1.0f - cell.fx, cell.fx};
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            if (!((corners >> c) & 1u)) continue;
                            // a corner the cell does not have (its code and the list entry disagree) adds nothing
                            const float w = ((cell.mask >> c) & 1u) ? wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1] : 0.0f;
                            const int idx = bk_a_index(((rt + (c >> 2)) * kKbY + ry + ((c >> 1) & 1)) * kKbX + rx + (c & 1), ql);
                            if (DSA3D_IN_RANGE(pr, at, static_cast<long long>(pr.blk_cap) * 8, 14))
                                out[at] = make_uint4(static_cast<uint32_t>(idx), __float_as_uint(w * cf[h].x), __float_as_uint(w * cf[h].y), 0u);
                            ++at;
                        }
                    }
                }
            }
            __threadfence_block();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_sorted[buf]));
            bk_named_barrier(4, kBkSorters);                            // the cursors are free for the next block
        }
    } else if (warp >= kStagerWarp0) {
        // ==================================================================== B operands: lane = query, warp = channel range
        constexpr int CPS = D / (kBkStagers / 32);                    // channels per warp
        constexpr int UPS = CPS / 8;                                  // 16-byte pieces of them
        const int sw = warp - kStagerWarp0;
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
        // where a chunk's entries lie, once its block has been sorted
        int sorted_seq = -1;
        auto locate_records = [&](const BkChunk& ch, int& n, const BkEntry*& recs) {
            n = 0; recs = my_sorted;
            if (!ch.valid) return;
            if (ch.seq != sorted_seq) {
                wait(&s.bar_sorted[ch.seq & 1], static_cast<uint32_t>((ch.seq >> 1) & 1), 38);
                sorted_seq = ch.seq;
            }
            const uint32_t b = *(volatile uint32_t*)&s.chunk_start[ch.seq & 1][ch.slot], e = *(volatile uint32_t*)&s.chunk_start[ch.seq & 1][ch.slot + 1];
            n = *abort_flag ? 0 : static_cast<int>(e - b);
            recs = my_sorted + static_cast<long long>(ch.seq & 1) * pr.blk_cap * 8 + b;
        };

        BkChunk ch;
        bk_start(ch);
        bk_advance(ch, wk, pr);
        int j = 0, prev_seq = -1, last_seq = -1, n_prev = 0;
        if (g == 1) {
            if (ch.valid) prev_seq = ch.seq;
            bk_advance(ch, wk, pr);
            j = 1;
        }
        int n = 0;
        const BkEntry* recs = my_sorted;
        BkEntry held[kBkHeld];
        locate_records(ch, n, recs);
#pragma unroll
        for (int h = 0; h < kBkHeld; ++h)
            if (gt + h * kBkGroup < n) held[h] = __ldcg(recs + gt + h * kBkGroup);
        for (int i = 0; ch.valid; ++i, j += 2) {
            bool drained = false;
            // ---- the group's previous chunk has been multiplied: its entries of A back to zero (and a finished block out)
            if (i >= 1) wait(&s.bar_done[g], static_cast<uint32_t>((i - 1) & 1), 33);
            if (j > 0 && ch.seq != prev_seq) {
                wait(&s.bar_done[g ^ 1], static_cast<uint32_t>(((j - 1) >> 1) & 1), 32);
                if (*(volatile uint32_t*)&s.blk_data[prev_seq & 1]) epilogue(prev_seq);
                drained = true;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (n_prev > kBkListCap) {
                float4* a = reinterpret_cast<float4*>(a_k);                  // the dK and dV matrices are adjacent
                for (int e = gt; e < 2 * kBkRows * kBkChunkQ / 4; e += kBkGroup) a[e] = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                const uint16_t* prev = s.list[g][(i - 1) & 1];
                for (int e = gt; e < n_prev; e += kBkGroup) { const int idx = prev[e]; a_k[idx] = 0.0f; a_v[idx] = 0.0f; }
            }
            bk_named_barrier(bar_id, kBkGroup);
            if (drained && gt == 0) {
                *(volatile uint32_t*)&s.blk_data[prev_seq & 1] = 0u;
                mbar_arrive(smem_u32(&s.bar_free[prev_seq & 1]));          // the sorters may reuse that block's buffers
            }
            // ---- this chunk's coefficients into A
            uint16_t* lst = s.list[g][i & 1];
#pragma unroll
            for (int h = 0; h < kBkHeld; ++h)
                if (gt + h * kBkGroup < n) {
                    atomicAdd(a_k + held[h].x, __uint_as_float(held[h].y));
                    atomicAdd(a_v + held[h].x, __uint_as_float(held[h].z));
                    lst[gt + h * kBkGroup] = static_cast<uint16_t>(held[h].x);
                }
            for (int base = kBkHeld * kBkGroup; base < n; base += kBkHeld * kBkGroup) {
#pragma unroll
                for (int h = 0; h < kBkHeld; ++h)
                    if (base + gt + h * kBkGroup < n) held[h] = __ldcg(recs + base + gt + h * kBkGroup);
#pragma unroll
                for (int h = 0; h < kBkHeld; ++h)
                    if (base + gt + h * kBkGroup < n) {
                        atomicAdd(a_k + held[h].x, __uint_as_float(held[h].y));
                        atomicAdd(a_v + held[h].x, __uint_as_float(held[h].z));
                        if (base + gt + h * kBkGroup < kBkListCap) lst[base + gt + h * kBkGroup] = static_cast<uint16_t>(held[h].x);
                    }
            }
            if (gt == 0) *(volatile uint32_t*)&s.count[g][i & 1] = static_cast<uint32_t>(n);
            fence_async_smem();                                       // the MMAs read A through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.bar_a_full[g]));
            // ---- the group's next chunk: its entries on their way
            last_seq = ch.seq;
            n_prev = n;
            bk_advance(ch, wk, pr);
            prev_seq = ch.valid ? ch.seq : -1;                        // block of the chunk between this one and the group's next
            bk_advance(ch, wk, pr);
            locate_records(ch, n, recs);
#pragma unroll
            for (int h = 0; h < kBkHeld; ++h)
                if (gt + h * kBkGroup < n) held[h] = __ldcg(recs + gt + h * kBkGroup);
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

template <int D>
cudaError_t launch_blocks_t(const void* q, const void* dout, const float* offsets, const float2* coef, float* acc_dk,
                            float* acc_dv, BkEntry* sorted, int total, int per_head, int by_count, int bx_count, int tb_begin,
                            int f0, int f1, int* flag, const Problem& pr, cudaStream_t stream) {
    auto kern = dkdv_block_kernel<D>;
    const size_t smem = sizeof(BkSmem<D>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (sms > kBkMaxCtas) sms = kBkMaxCtas;
    const unsigned grid = static_cast<unsigned>(total < sms ? total : sms);     // persistent: one CTA per SM
    kern<<<grid, kBkThreads, smem, stream>>>(static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(dout),
                                             offsets, coef, acc_dk, acc_dv, sorted, total, per_head, by_count, bx_count,
                                             tb_begin, f0, f1, flag, pr);
    return cudaGetLastError();
}

}  // namespace

KeyBlockLayout key_block_layout(const Problem& pr) {
    KeyBlockLayout kb{};
    kb.blocks = static_cast<long long>((pr.T + kKbT - 1) / kKbT) * ((pr.H + kKbY - 1) / kKbY) * ((pr.W + kKbX - 1) / kKbX) * pr.heads;
    // a block of 256 keys is touched by 256 * P samples, each counted for about 1.6 blocks; the rest of the
    // room is for the blocks that get more than their share (a sample that finds a list full is scattered directly)
    kb.cap = (kBkRows * pr.P * 9 / 5 + 255) / 256 * 256;
    kb.count_bytes = (static_cast<size_t>(kb.blocks) * sizeof(uint32_t) + 255) & ~static_cast<size_t>(255);
    kb.list_bytes = static_cast<size_t>(kb.blocks) * kb.cap * sizeof(uint32_t);
    kb.sorted_bytes = static_cast<size_t>(kBkMaxCtas) * 2 * kb.cap * 8 * sizeof(BkEntry);       // up to eight entries per listed sample
    return kb;
}

bool key_blocks_shape_covered(const Problem& pr) {
    if (pr.d != 128 && pr.d != 64) return false;
    if (pr.P > 256) return false;                                                     // 8-bit sample field of a list entry
    const long long blocks = static_cast<long long>((pr.T + kKbT - 1) / kKbT) * ((pr.H + kKbY - 1) / kKbY) *
                             ((pr.W + kKbX - 1) / kKbX) * pr.heads;
    return blocks < (1LL << 30);
}

cudaError_t launch_dkdv_blocks(const void* q, const void* dout, const float* offsets, const float2* coef, float* acc_dk,
                               float* acc_dv, const Problem& pr, cudaStream_t stream) {
    if (!key_blocks_shape_covered(pr) || !pr.blk_count || !pr.blk_list) return cudaErrorInvalidValue;
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
    const KeyBlockLayout kb = key_block_layout(pr);
    BkEntry* sorted = reinterpret_cast<BkEntry*>(reinterpret_cast<char*>(pr.blk_list) + kb.list_bytes);
#define DSA3D_BK(DD) launch_blocks_t<DD>(q, dout, offsets, coef, acc_dk, acc_dv, sorted, total, per_head, by_count, bx_count, \
                                         tb_begin, f0, f1, flag, pr, stream)
    return pr.d == 128 ? DSA3D_BK(128) : DSA3D_BK(64);
#undef DSA3D_BK
}

}  // namespace dsa3d
