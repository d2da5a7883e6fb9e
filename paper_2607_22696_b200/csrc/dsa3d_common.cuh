// Shared device helpers of the 3D-DSA kernels: problem description, element access for
// fp32 / bf16 storage, sample geometry (Formulation: position = token coordinate + window
// displacement + learned offset; trilinear corners with zero padding) and group shuffles.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsa3d {

// One contribution to dK/dV as the tile kernel bins it: byte offset of the query's q/dO row
// pair in shared memory and the two coefficients (w_c * ck_p, w_c * cv_p).
using TileEntry = uint4;            // {offset, fp32 wk, fp32 wv, unused}

struct Problem {
    int T, H, W, heads, d;
    int kt, kh, kw, P;
    // ceil(2^20 / kw) and ceil(2^20 / kh): p / kw = (p * inv_kw) >> 20 exactly for p < 2^8 (P <= 256), so that
    // a sample's window cell needs no integer division
    unsigned inv_kw, inv_kh;
    long long N;       // T*H*W
    long long items;   // work items of this launch: one per (query token, head) = q_count*heads
    // Query tokens [q_begin, q_begin + q_count) are processed (the whole grid unless a caller
    // works through the video in slabs of frames); K and V always cover the whole grid.
    long long q_begin, q_count;
    // Query tiling of the backward scatter (tile_t < 1: no tiling, every dK/dV contribution
    // goes straight to the global accumulators).  A corner is "in the halo" of a query when
    // it lies within `halo` grid cells of the query's tile on every axis.
    int tile_t, tile_y, tile_x, halo;
    int tiles_t, tiles_y, tiles_x;
    int tt_begin, tt_count;   // tile rows along t that the tile kernel visits (all: 0, tiles_t)
    // Key-block scheme (see block_near_mask below) instead of query tiles: the gather kernel appends every
    // sample to the list of each key block one of its corners lies in (blk_list [blocks][blk_cap] of packed
    // entries, blk_count [blocks], blocks numbered ((head * tb + bt) * by + by_) * bx + bx_ over the whole
    // grid) and scatters only the corners whose query lies outside the region of the corner's key block - or
    // whose block's list was full.
    int key_blocks;
    uint32_t* blk_count;
    uint32_t* blk_list;
    int blk_cap;
    // Checked build (-DDSA3D_DEBUG) only: device word that receives the first out-of-range index a
    // kernel was about to use (0 = none); NULL otherwise.
    unsigned long long* debug_word;
    // Backward behind a check of the offsets (dsa3d_backward_bounded_offsets): the general kernels run only
    // if this device word is non-zero (the check found offsets its tile kernels do not cover); NULL: always.
    const int* gate;
};

// True when a gated general kernel has nothing to do (see Problem::gate).
__device__ __forceinline__ bool gated_off(const Problem& pr) { return pr.gate != nullptr && *pr.gate == 0; }

// Checked build: every row a gather reads and every row or bin a scatter writes is tested against its
// tensor's extent first; a violation is recorded (first one wins: code in the top 8 bits, the offending
// element offset in the rest) and the access is skipped - nothing traps.  In the normal build the
// tests compile to `true`.
#ifdef DSA3D_DEBUG
__device__ __forceinline__ bool debug_in_range(const Problem& pr, long long offset, long long extent, int code) {
    if (offset >= 0 && offset < extent) return true;
    if (pr.debug_word)
        atomicCAS(pr.debug_word, 0ull, (static_cast<unsigned long long>(code) << 56) |
                                           (static_cast<unsigned long long>(offset) & ((1ull << 56) - 1)));
    return false;
}
#define DSA3D_IN_RANGE(pr, offset, extent, code) dsa3d::debug_in_range((pr), (offset), (extent), (code))
#else
#define DSA3D_IN_RANGE(pr, offset, extent, code) true
#endif

// ---------------------------------------------------------------------------------------
// Element access.  A lane handles NV consecutive 16-byte vectors of a row (8 bf16 or 4 fp32
// channels each).
// `Row` keeps that vector in its storage form.  For bf16 the dot products (both factors
// bf16) use the sm_100 mixed-precision instruction fma.rn.f32.bf16 (exact fp32 product,
// fp32 accumulate), which needs no unpacking; `axpy` (fp32 coefficient) widens the row.
// ---------------------------------------------------------------------------------------
// Two independent fp32 FMAs in one instruction (sm_100 fma.rn.f32x2): a0 += x0*y0, a1 += x1*y1,
// each rounded exactly as fmaf would.  Pays where a loop is bound by issue slots and most of its
// instructions are FMAs.
__device__ __forceinline__ void fma2(float& a0, float& a1, float x0, float x1, float y0, float y1) {
    unsigned long long acc, x, y;
    asm("mov.b64 %0, {%1, %2};" : "=l"(acc) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "f"(x0), "f"(x1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(y) : "f"(y0), "f"(y1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(x), "l"(y));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc));
}

// The 128-channel backward gather (two 16-byte vectors per lane) uses the packed FMA in its row
// scalings (2.9 % faster); the forward and the narrower kernels measured no gain and keep fmaf.
constexpr bool kPackedAxpy = true;

template <typename T, int NV> struct Elt;       // NV = 16-byte vectors per lane (1 or 2)

template <int NV> struct Elt<float, NV> {
    static constexpr int VEC = 4 * NV;
    struct Row { float v[VEC]; };
    static __device__ __forceinline__ Row load(const float* p) {
        Row r;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const float4 x = __ldg(reinterpret_cast<const float4*>(p) + i);
            r.v[4 * i] = x.x; r.v[4 * i + 1] = x.y; r.v[4 * i + 2] = x.z; r.v[4 * i + 3] = x.w;
        }
        return r;
    }
    static __device__ __forceinline__ Row zero() {
        Row r;
#pragma unroll
        for (int e = 0; e < VEC; ++e) r.v[e] = 0.0f;
        return r;
    }
    static __device__ __forceinline__ float dot(const Row& a, const Row& b, float acc) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc = fmaf(a.v[e], b.v[e], acc);
        return acc;
    }
    static __device__ __forceinline__ void axpy(float c, const Row& x, float (&acc)[VEC]) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] = fmaf(c, x.v[e], acc[e]);
    }
    static __device__ __forceinline__ void axpy_paired(float c, const Row& x, float (&acc)[VEC]) { axpy(c, x, acc); }
    static __device__ __forceinline__ void to_float(const Row& x, float (&f)[VEC]) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] = x.v[e];
    }
    static __device__ __forceinline__ void store(float* p, const float (&x)[VEC]) {
#pragma unroll
        for (int i = 0; i < NV; ++i)
            reinterpret_cast<float4*>(p)[i] = make_float4(x[4 * i], x[4 * i + 1], x[4 * i + 2], x[4 * i + 3]);
    }
};

__device__ __forceinline__ float fma_bf16(unsigned short a, unsigned short b, float c) {
    float d;
    asm("fma.rn.f32.bf16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
    return d;
}

__device__ __forceinline__ void split_b32(uint32_t r, unsigned short& lo, unsigned short& hi) {
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(r));
}

template <int NV> struct Elt<__nv_bfloat16, NV> {
    static constexpr int VEC = 8 * NV;
    static constexpr int NW = 4 * NV;            // 32-bit words per lane
    struct Row { uint32_t w[NW]; };
    static __device__ __forceinline__ Row load(const __nv_bfloat16* p) {
        Row r;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(p) + i);
            r.w[4 * i] = x.x; r.w[4 * i + 1] = x.y; r.w[4 * i + 2] = x.z; r.w[4 * i + 3] = x.w;
        }
        return r;
    }
    static __device__ __forceinline__ Row zero() {
        Row r;
#pragma unroll
        for (int i = 0; i < NW; ++i) r.w[i] = 0u;
        return r;
    }
    static __device__ __forceinline__ float dot(const Row& a, const Row& b, float acc) {
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            unsigned short al, ah, bl, bh;
            split_b32(a.w[i], al, ah);
            split_b32(b.w[i], bl, bh);
            acc = fma_bf16(al, bl, acc);
            acc = fma_bf16(ah, bh, acc);
        }
        return acc;
    }
    // acc += c * x with an fp32 coefficient: the bf16 values are widened (one shift or mask
    // each) and multiplied in fp32, so the coefficient keeps all its bits.  (Rounding the
    // coefficient to bf16 and using the mixed instruction was measured 12 % faster overall, but
    // its error reaches the 2e-2 bound on rare elements of very large tensors.)
    static __device__ __forceinline__ void axpy(float c, const Row& x, float (&acc)[VEC]) {
        if constexpr (NV == 2 && kPackedAxpy) {
#pragma unroll
            for (int i = 0; i < NW; ++i)
                fma2(acc[2 * i], acc[2 * i + 1], c, c, __uint_as_float(x.w[i] << 16), __uint_as_float(x.w[i] & 0xffff0000u));
        } else {
#pragma unroll
            for (int i = 0; i < NW; ++i) {
                acc[2 * i] = fmaf(c, __uint_as_float(x.w[i] << 16), acc[2 * i]);
                acc[2 * i + 1] = fmaf(c, __uint_as_float(x.w[i] & 0xffff0000u), acc[2 * i + 1]);
            }
        }
    }
    // The same with two FMAs per instruction whatever the lane width (for loops that are bound by issue slots).
    static __device__ __forceinline__ void axpy_paired(float c, const Row& x, float (&acc)[VEC]) {
#pragma unroll
        for (int i = 0; i < NW; ++i)
            fma2(acc[2 * i], acc[2 * i + 1], c, c, __uint_as_float(x.w[i] << 16), __uint_as_float(x.w[i] & 0xffff0000u));
    }
    static __device__ __forceinline__ void to_float(const Row& x, float (&f)[VEC]) {
#pragma unroll
        for (int i = 0; i < NW; ++i) {          // bf16 is the upper half of an fp32
            f[2 * i] = __uint_as_float(x.w[i] << 16);
            f[2 * i + 1] = __uint_as_float(x.w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[VEC]) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(x[8 * i + 2 * j], x[8 * i + 2 * j + 1]);   // RNE
                w[j] = *reinterpret_cast<const uint32_t*>(&h);
            }
            reinterpret_cast<uint4*>(p)[i] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
};

// ---------------------------------------------------------------------------------------
// Sample geometry.  (it, iy, ix) is corner (0,0,0) of the cell (a component may be -1;
// only corners flagged in `mask` are ever dereferenced), bit c = ct*4 + cy*2 + cx of
// `mask` says corner c lies inside the grid, f* are the fractional parts.  A sample with a
// NaN position or one at < -1 or >= size on any axis has mask 0.  The position is
// float(coord + b) + offset with one fp32 rounding, then floorf, then the fp32 difference:
// the same sequence on every path so that the integer cell decision never depends on who
// computes it.
// ---------------------------------------------------------------------------------------
struct Cell {
    int it, iy, ix;
    unsigned mask;
    float ft, fy, fx;
};

// What a lane needs to process a sample somebody else located: linear index of corner
// (0,0,0), corner mask, fractional parts.
struct Sample {
    int base;
    unsigned mask;
    float ft, fy, fx;
};

__device__ __forceinline__ bool axis_cell(int coord_plus_b, float off, int size, int& i0, float& f) {
    const float pi = __fadd_rn(static_cast<float>(coord_plus_b), off);
    if (!(pi >= -1.0f) || !(pi < static_cast<float>(size))) return false;
    const float fl = floorf(pi);
    i0 = static_cast<int>(fl);
    f = __fsub_rn(pi, fl);
    return true;
}

// Bit c of the result is set when corner c = (ct, cy, cx) has lo <= i0 + c < hi on every axis,
// where the test per axis is written as an unsigned range check on (i0 - lo).
__device__ __forceinline__ unsigned corner_mask(int rt, int ry, int rx, int et, int ey, int ex) {
    const unsigned t0 = static_cast<unsigned>(rt) < static_cast<unsigned>(et);
    const unsigned t1 = static_cast<unsigned>(rt + 1) < static_cast<unsigned>(et);
    const unsigned y0 = static_cast<unsigned>(ry) < static_cast<unsigned>(ey);
    const unsigned y1 = static_cast<unsigned>(ry + 1) < static_cast<unsigned>(ey);
    const unsigned x0 = static_cast<unsigned>(rx) < static_cast<unsigned>(ex);
    const unsigned x1 = static_cast<unsigned>(rx + 1) < static_cast<unsigned>(ex);
    const unsigned yx = (y0 & x0) | ((y0 & x1) << 1) | ((y1 & x0) << 2) | ((y1 & x1) << 3);
    return (t0 ? yx : 0u) | (t1 ? (yx << 4) : 0u);
}

// The same from the three offset components already loaded.
__device__ __forceinline__ Cell make_cell_values(const Problem& pr, int t, int y, int x, int p, float ot, float oy,
                                                 float ox) {
    const int pk = static_cast<int>((static_cast<unsigned>(p) * pr.inv_kw) >> 20);      // p / kw
    const int w = p - pk * pr.kw;
    const int u = static_cast<int>((static_cast<unsigned>(pk) * pr.inv_kh) >> 20);     // p / (kw * kh)
    const int v = pk - u * pr.kh;
    Cell c;
    c.it = c.iy = c.ix = 0;
    c.mask = 0u;
    c.ft = c.fy = c.fx = 0.0f;
    int it, iy, ix;
    float ft, fy, fx;
    if (!axis_cell(t + u - pr.kt / 2, ot, pr.T, it, ft)) return c;
    if (!axis_cell(y + v - pr.kh / 2, oy, pr.H, iy, fy)) return c;
    if (!axis_cell(x + w - pr.kw / 2, ox, pr.W, ix, fx)) return c;
    c.it = it; c.iy = iy; c.ix = ix;
    c.ft = ft; c.fy = fy; c.fx = fx;
    c.mask = corner_mask(it, iy, ix, pr.T, pr.H, pr.W);
    return c;
}

__device__ __forceinline__ Cell make_cell(const Problem& pr, int t, int y, int x, int p,
                                          const float* __restrict__ off3) {
    const int pk = static_cast<int>((static_cast<unsigned>(p) * pr.inv_kw) >> 20);      // p / kw
    const int w = p - pk * pr.kw;
    const int u = static_cast<int>((static_cast<unsigned>(pk) * pr.inv_kh) >> 20);     // p / (kw * kh)
    const int v = pk - u * pr.kh;
    Cell c;
    c.it = c.iy = c.ix = 0;
    c.mask = 0u;
    c.ft = c.fy = c.fx = 0.0f;
    int it, iy, ix;
    float ft, fy, fx;
    const float ot = __ldg(off3), oy = __ldg(off3 + 1), ox = __ldg(off3 + 2);
    if (!axis_cell(t + u - pr.kt / 2, ot, pr.T, it, ft)) return c;
    if (!axis_cell(y + v - pr.kh / 2, oy, pr.H, iy, fy)) return c;
    if (!axis_cell(x + w - pr.kw / 2, ox, pr.W, ix, fx)) return c;
    c.it = it; c.iy = iy; c.ix = ix;
    c.ft = ft; c.fy = fy; c.fx = fx;
    c.mask = corner_mask(it, iy, ix, pr.T, pr.H, pr.W);
    return c;
}

__device__ __forceinline__ Sample to_sample(const Problem& pr, const Cell& c) {
    Sample s;
    s.base = (c.it * pr.H + c.iy) * pr.W + c.ix;
    s.mask = c.mask;
    s.ft = c.ft; s.fy = c.fy; s.fx = c.fx;
    return s;
}

// Corners of `c` that lie in the halo box of the tile containing query (t, y, x).
__device__ __forceinline__ unsigned halo_corner_mask(const Problem& pr, const Cell& c, int t, int y, int x) {
    if (pr.tile_t < 1) return 0u;
    const int lo_t = (t / pr.tile_t) * pr.tile_t - pr.halo;
    const int lo_y = (y / pr.tile_y) * pr.tile_y - pr.halo;
    const int lo_x = (x / pr.tile_x) * pr.tile_x - pr.halo;
    return corner_mask(c.it - lo_t, c.iy - lo_y, c.ix - lo_x, pr.tile_t + 2 * pr.halo,
                       pr.tile_y + 2 * pr.halo, pr.tile_x + 2 * pr.halo);
}

// ---------------------------------------------------------------------------------------
// Key blocks (the tensor-core dK/dV kernel, dsa3d_backward_blocks.cu).  The grid is cut into
// blocks of 4 x 8 x 8 key positions; the kernel that owns a block sums the contributions of every
// query in the block's REGION: 16 frames from t0 - 6, 20 rows from y0 - 6 (five strips of 4),
// 24 columns from x0 - 8 (three strips of 8).  A contribution whose query lies outside the
// region of its key's block is scattered by the gather kernel itself.
// ---------------------------------------------------------------------------------------
constexpr int kKbT = 4, kKbY = 8, kKbX = 8;
constexpr int kKbLoT = 6, kKbLoY = 6, kKbLoX = 8;             // the region starts this far below the block
constexpr int kKbRegT = 16, kKbRegY = 20, kKbRegX = 24;       // its extent

// Bit c is set when the query (t, y, x) lies in the region of the key block holding corner c of the cell.
__device__ __forceinline__ unsigned block_near_mask(const Cell& c, int t, int y, int x) {
    unsigned nt[2], ny[2], nx[2];
#pragma unroll
    for (int a = 0; a < 2; ++a) {
        nt[a] = static_cast<unsigned>(t - ((c.it + a) & ~(kKbT - 1)) + kKbLoT) < static_cast<unsigned>(kKbRegT);
        ny[a] = static_cast<unsigned>(y - ((c.iy + a) & ~(kKbY - 1)) + kKbLoY) < static_cast<unsigned>(kKbRegY);
        nx[a] = static_cast<unsigned>(x - ((c.ix + a) & ~(kKbX - 1)) + kKbLoX) < static_cast<unsigned>(kKbRegX);
    }
    const unsigned yx = (ny[0] & nx[0]) | ((ny[0] & nx[1]) << 1) | ((ny[1] & nx[0]) << 2) | ((ny[1] & nx[1]) << 3);
    return (nt[0] ? yx : 0u) | (nt[1] ? (yx << 4) : 0u);
}

// Entry of a key block's sample list: chunk slot of the query in the block's region (8 bits), query inside the
// chunk (5), sample (8), corner (0,0,0) of the cell relative to the block + 1 (3 + 4 + 4 bits).
__device__ __forceinline__ uint32_t block_entry(int slot, int ql, int p, int rt1, int ry1, int rx1) {
    return static_cast<uint32_t>(slot) | (static_cast<uint32_t>(ql) << 8) | (static_cast<uint32_t>(p) << 13) |
           (static_cast<uint32_t>(rt1) << 21) | (static_cast<uint32_t>(ry1) << 24) | (static_cast<uint32_t>(rx1) << 28);
}
constexpr int kKbChunkY = 4, kKbChunkX = 8;                    // a chunk of the region: 4 rows x 8 columns of one frame
constexpr int kKbChunksX = kKbRegX / kKbChunkX, kKbChunksPerFrame = (kKbRegY / kKbChunkY) * kKbChunksX;   // 3, 15

// The gather kernel's side of the key-block scheme for one sample: append it to the list of every block that
// holds one of its corners and whose region holds the query; return the corners left for the direct scatter.
__device__ __forceinline__ unsigned block_lists_append(const Problem& pr, const Cell& c, int t, int y, int x, int m, int p) {
    const unsigned near = block_near_mask(c, t, y, x) & c.mask;
    unsigned far = c.mask & ~near;
    if (near == 0u) return far;
    const int bt_n = (pr.T + kKbT - 1) / kKbT, by_n = (pr.H + kKbY - 1) / kKbY, bx_n = (pr.W + kKbX - 1) / kKbX;
    // along an axis the two corners lie in different blocks only when the second one starts a block
    const unsigned cross = (((c.it + 1) & (kKbT - 1)) == 0 ? 1u : 0u) | (((c.iy + 1) & (kKbY - 1)) == 0 ? 2u : 0u) |
                           (((c.ix + 1) & (kKbX - 1)) == 0 ? 4u : 0u);
    for (unsigned sel = 0; sel < 8u; ++sel) {
        if (sel & ~cross) continue;
        // corners of this block: second corner along the crossing axes chosen by `sel`, both along the others
        unsigned sub = 0xffu;
        if (cross & 1u) sub &= (sel & 1u) ? 0xf0u : 0x0fu;
        if (cross & 2u) sub &= (sel & 2u) ? 0xccu : 0x33u;
        if (cross & 4u) sub &= (sel & 4u) ? 0xaau : 0x55u;
        sub &= near;
        if (sub == 0u) continue;
        const int t0 = (c.it + static_cast<int>(sel & 1u)) & ~(kKbT - 1), y0 = (c.iy + static_cast<int>((sel >> 1) & 1u)) & ~(kKbY - 1),
                  x0 = (c.ix + static_cast<int>((sel >> 2) & 1u)) & ~(kKbX - 1);
        const long long bid = ((static_cast<long long>(m) * bt_n + t0 / kKbT) * by_n + y0 / kKbY) * bx_n + x0 / kKbX;
        const int dy = y - (y0 - kKbLoY), dx = x - (x0 - kKbLoX);
        const int slot = ((t - (t0 - kKbLoT)) * (kKbRegY / kKbChunkY) + dy / kKbChunkY) * kKbChunksX + dx / kKbChunkX;
        const uint32_t entry = block_entry(slot, (dy % kKbChunkY) * kKbChunkX + dx % kKbChunkX, p, c.it - t0 + 1, c.iy - y0 + 1, c.ix - x0 + 1);
        const uint32_t at = atomicAdd(pr.blk_count + bid, 1u);
        if (at < static_cast<uint32_t>(pr.blk_cap)) pr.blk_list[bid * pr.blk_cap + at] = entry;
        else far |= sub;                                      // list full: these corners go the direct way
    }
    return far;
}

// Shuffles inside a group of LPR consecutive lanes (LPR a power of two <= 32).
template <int LPR> __device__ __forceinline__ unsigned group_mask(int lane) {
    if constexpr (LPR == 32) {
        return 0xffffffffu;
    } else {
        return ((1u << LPR) - 1u) << (lane & ~(LPR - 1));
    }
}

// All shuffles below name the full warp: the kernels keep every lane of a warp alive and
// on the same control path at each shuffle (a group past the end of the problem repeats
// the last item with its stores switched off), so no per-group mask is needed.
constexpr unsigned kFullMask = 0xffffffffu;

template <int LPR> __device__ __forceinline__ float group_sum(float v, unsigned gmask) {
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(gmask, v, o, LPR);
    return v;
}

// Sum 8 per-lane numbers over the group so that every sum ends up on some lane, with a
// quarter of the shuffles a butterfly per value would take: at each of the first three
// xor distances a lane hands half of its values to its partner and keeps the other half.
// On return v[0] of lane gl holds the complete sum number reduce8_index<LPR>(gl).
// (LPR >= 8; narrower groups use group_sum.)
template <int LPR> __device__ __forceinline__ int reduce8_index(int gl) {
    return (((gl / (LPR / 2)) & 1) << 2) | (((gl / (LPR / 4)) & 1) << 1) | ((gl / (LPR / 8)) & 1);
}
template <int LPR> __device__ __forceinline__ int reduce8_lane(int index) {     // a lane holding sum `index`
    return ((index >> 2) & 1) * (LPR / 2) + ((index >> 1) & 1) * (LPR / 4) + (index & 1) * (LPR / 8);
}
template <int LPR> __device__ __forceinline__ void group_reduce8(float (&v)[8], int gl, unsigned gmask) {
    static_assert(LPR >= 8, "needs three halving steps");
    int n = 8;
#pragma unroll
    for (int d = LPR / 2; d >= LPR / 8; d >>= 1) {
        const bool upper = (gl & d) != 0;
        n >>= 1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i < n) {
                const float send = upper ? v[i] : v[i + n];
                const float keep = upper ? v[i + n] : v[i];
                v[i] = keep + __shfl_xor_sync(gmask, send, d, LPR);
            }
        }
    }
#pragma unroll
    for (int d = LPR / 16; d > 0; d >>= 1) v[0] += __shfl_xor_sync(gmask, v[0], d, LPR);
}

// Value and the three partial derivatives (along t, y, x) of the trilinear interpolant of
// eight corner numbers a[c], c = ct*4 + cy*2 + cx, at fractional position (ft, fy, fx):
// value = sum_c w_c a_c, d/da = sum_c (dw_c/da) a_c.  Corners outside the grid enter as 0.
__device__ __forceinline__ void trilerp_grad(const float (&a)[8], float ft, float fy, float fx, float& val,
                                             float& dt, float& dy, float& dx) {
    float L[4], X[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        X[i] = a[2 * i + 1] - a[2 * i];
        L[i] = fmaf(fx, X[i], a[2 * i]);
    }
    float M[2], Y[2], Xy[2];
#pragma unroll
    for (int ct = 0; ct < 2; ++ct) {
        Y[ct] = L[2 * ct + 1] - L[2 * ct];
        M[ct] = fmaf(fy, Y[ct], L[2 * ct]);
        Xy[ct] = fmaf(fy, X[2 * ct + 1] - X[2 * ct], X[2 * ct]);
    }
    dt = M[1] - M[0];
    val = fmaf(ft, dt, M[0]);
    dy = fmaf(ft, Y[1] - Y[0], Y[0]);
    dx = fmaf(ft, Xy[1] - Xy[0], Xy[0]);
}

template <int LPR> __device__ __forceinline__ Sample group_bcast(const Sample& s, int src, unsigned gmask) {
    Sample r;
    r.base = __shfl_sync(gmask, s.base, src, LPR);
    r.mask = __shfl_sync(gmask, s.mask, src, LPR);
    r.ft = __shfl_sync(gmask, s.ft, src, LPR);
    r.fy = __shfl_sync(gmask, s.fy, src, LPR);
    r.fx = __shfl_sync(gmask, s.fx, src, LPR);
    return r;
}

// One 16-byte fp32 reduction into global memory (the dK/dV accumulators).
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace dsa3d
