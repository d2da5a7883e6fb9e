// Backward for learned offsets below 1 in size on every axis (window (3,3,3), bf16, 64 or 128 channels): the
// regime in which the offsets are perturbations of the fixed window (Formulation).  Every corner of every
// sample of a query then lies in the box of 5 x 5 x 5 grid positions around the query, so nothing has to be
// gathered or scattered row by row:
//
//   1. fixed_window_tables_kernel (instance (5,5,5)) leaves, per (query, head), the dot products
//      a_j = q . K_j and b_j = dO . V_j of the 6 x 6 x 6 positions from query - 2 (dense Q.K^T and dO.V^T
//      tiles on the tensor cores).  The sixth position per axis is the +1 neighbour that the one-sided
//      derivative reads when an offset just below +1 rounds the fp32 position up to a grid position.
//   2. bounded_offsets_backward_query_kernel (this file): per sample the cell and fractions exactly as the
//      general kernel forms them, the logit, g = dO . V(sample) and their derivatives along the three axes as
//      trilinear combinations of eight table entries; alpha from the forward's lse, delta, dS, dOffsets; the
//      coefficients  scale dS_p w_c  and  alpha_p w_c  of the eight corners summed per box position into a
//      5 x 5 x 5 box of ck and cv, which go out as planes [head][125][token] (bf16 head | remainder words).
//   3. fixed_window_planes_grad_kernel (instance (5,5,5)):  dQ, dK, dV are the three weighted sums of a
//      fixed (5,5,5) window with those coefficients, plane-by-plane products on the tensor cores.
//
// All of it runs behind a device check of the offsets (finite, |offset| < 1 everywhere -> gate word 0): the
// three kernels do nothing unless the gate is 0, the general backward kernels, queued behind them, nothing
// unless it is 1 - the call stays asynchronous and is right for any offsets.
#include <cuda_bf16.h>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"

namespace dsa3d {
namespace {

constexpr int kBoLanes = 8;                  // lanes per (query, head): the eight corners of a sample in the last phase
constexpr int kBoThreads = 128;
constexpr int kBoGroups = kBoThreads / kBoLanes;
constexpr int kBoP = 27;                     // window (3,3,3)
constexpr int kBoTab = 6, kBoTabCells = kBoTab * kBoTab * kBoTab;      // table box (from query - 2)
constexpr int kBoBox = 5, kBoBoxCells = kBoBox * kBoBox * kBoBox;      // coefficient box (from query - 2)
constexpr int kBoRounds = (kBoP + kBoLanes - 1) / kBoLanes;

struct BoGroup {
    union {                                  // the tables are read for the last time before the box is first written
        struct { float tab_a[kBoTabCells], tab_b[kBoTabCells]; };
        struct { float box_ck[kBoBoxCells], box_cv[kBoBoxCells]; };
    };
    float s_ck[kBoP], s_cv[kBoP], s_ft[kBoP], s_fy[kBoP], s_fx[kBoP];
    int s_cell[kBoP];                        // bt | by << 3 | bx << 6 of corner (0,0,0) in the coefficient box, -1: dead sample
};

// An fp32 value as two bf16 numbers whose sum is the value to 2^-17 relative: the nearest bf16 in the low
// half of the word, the nearest bf16 of what is left in the high half.
__device__ __forceinline__ uint32_t split_bf16_pair(float x) {
    const __nv_bfloat16 head = __float2bfloat16_rn(x);
    const __nv_bfloat16 rest = __float2bfloat16_rn(x - __bfloat162float(head));
    return static_cast<uint32_t>(__bfloat16_as_ushort(head)) | (static_cast<uint32_t>(__bfloat16_as_ushort(rest)) << 16);
}

__global__ void __launch_bounds__(kBoThreads)
bounded_offsets_backward_query_kernel(const float* __restrict__ offsets, const float* __restrict__ lse,
                                      const float* __restrict__ table, float* __restrict__ doffsets,
                                      uint32_t* __restrict__ planes, const int* __restrict__ gate, const Problem pr) {
    extern __shared__ __align__(16) unsigned char bo_raw[];
    if (gate != nullptr && *gate != 0) return;             // the general kernels take this call
    BoGroup& g = reinterpret_cast<BoGroup*>(bo_raw)[threadIdx.x / kBoLanes];
    const int gl = threadIdx.x & (kBoLanes - 1);
    const long long block_first = static_cast<long long>(blockIdx.x) * kBoGroups;
    long long item = block_first + threadIdx.x / kBoLanes;
    const bool active = item < pr.items;                   // a trailing group repeats the last item, stores off
    if (!active) item = pr.items - 1;
    const int m = static_cast<int>(item / pr.q_count);
    const long long n = pr.q_begin + (item - static_cast<long long>(m) * pr.q_count);
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const long long row = n * pr.heads + m;
    const float scale = rsqrtf(static_cast<float>(pr.d));
    const float lse2 = __ldg(lse + row) * kLog2e;

    // ---- the query's tables, the coefficient box cleared
    {
        const float* mine = table + row * (2 * kBoTabCells);
        for (int i = gl; i < kBoTabCells; i += kBoLanes) {
            g.tab_a[i] = __ldg(mine + i);
            g.tab_b[i] = __ldg(mine + kBoTabCells + i);
        }
    }
    __syncwarp();

    // ---- per sample (lanes over samples): logit, g, their derivatives; alpha; delta
    float alpha[kBoRounds], gp[kBoRounds], da[kBoRounds][3], db[kBoRounds][3];
    float delta = 0.0f;
    const float* off_row = offsets + row * (kBoP * 3);
#pragma unroll
    for (int r = 0; r < kBoRounds; ++r) {
        const int p = r * kBoLanes + gl;
        alpha[r] = gp[r] = 0.0f;
        da[r][0] = da[r][1] = da[r][2] = db[r][0] = db[r][1] = db[r][2] = 0.0f;
        if (p >= kBoP) continue;
        const Cell cell = make_cell_values(pr, t, y, x, p, __ldg(off_row + p * 3), __ldg(off_row + p * 3 + 1), __ldg(off_row + p * 3 + 2));
        float sdot = 0.0f;
        int code = -1;
        if (cell.mask != 0u) {
            // corner (0,0,0) relative to query - 2: 0 .. 4 on every axis while the offsets are below 1 in size
            // (the clamp keeps a garbage offset, which the gate excludes, from indexing outside the tables)
            const int bt = min(max(cell.it - (t - 2), 0), kBoTab - 2), by = min(max(cell.iy - (y - 2), 0), kBoTab - 2),
                      bx = min(max(cell.ix - (x - 2), 0), kBoTab - 2);
            const int at = (bt * kBoTab + by) * kBoTab + bx;
            float a[8], b[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int i = at + ((c >> 2) * kBoTab + ((c >> 1) & 1)) * kBoTab + (c & 1);
                a[c] = g.tab_a[i];                      // positions outside the grid hold 0: the zero-padded key
                b[c] = g.tab_b[i];
            }
            trilerp_grad(a, cell.ft, cell.fy, cell.fx, sdot, da[r][0], da[r][1], da[r][2]);
            trilerp_grad(b, cell.ft, cell.fy, cell.fx, gp[r], db[r][0], db[r][1], db[r][2]);
            code = bt | (by << 3) | (bx << 6);
        }
        alpha[r] = exp2f(fmaf(sdot, scale * kLog2e, -lse2));   // a dead sample stays in the softmax with logit 0
        delta = fmaf(alpha[r], gp[r], delta);
        g.s_cell[p] = code;
        g.s_ft[p] = cell.ft; g.s_fy[p] = cell.fy; g.s_fx[p] = cell.fx;
    }
    delta = group_sum<kBoLanes>(delta, kFullMask);

    // ---- dS, dOffsets, the two coefficients of every sample
#pragma unroll
    for (int r = 0; r < kBoRounds; ++r) {
        const int p = r * kBoLanes + gl;
        if (p >= kBoP) continue;
        const float ck = scale * alpha[r] * (gp[r] - delta);
        g.s_ck[p] = ck;
        g.s_cv[p] = alpha[r];
        if (active) {
            float* dst = doffsets + (row * kBoP + p) * 3;
            dst[0] = fmaf(ck, da[r][0], alpha[r] * db[r][0]);
            dst[1] = fmaf(ck, da[r][1], alpha[r] * db[r][1]);
            dst[2] = fmaf(ck, da[r][2], alpha[r] * db[r][2]);
        }
    }
    __syncwarp();                                          // every table read of the group is done: the box takes their place
    for (int i = gl; i < kBoBoxCells; i += kBoLanes) g.box_ck[i] = g.box_cv[i] = 0.0f;
    __syncwarp();

    // ---- the coefficient box: sample after sample, the eight lanes taking the eight corners.  A lane takes
    //      the corner whose box position has the lane's parity pattern (t, y, x parities = the lane's three
    //      bits): the eight corners of a cell have the eight patterns once each, so a box position is only
    //      ever touched by one lane - plain read-add-write, no ordering between lanes, sums in sample order.
    {
#pragma unroll 3
        for (int p = 0; p < kBoP; ++p) {
            const int code = g.s_cell[p];
            if (code < 0) continue;
            const int bt = code & 7, by = (code >> 3) & 7, bx = code >> 6;
            const int ct = (gl >> 2) ^ (bt & 1), cy = ((gl >> 1) & 1) ^ (by & 1), cx = (gl & 1) ^ (bx & 1);
            const float ft = g.s_ft[p], fy = g.s_fy[p], fx = g.s_fx[p];
            const float w = (ct ? ft : 1.0f - ft) * (cy ? fy : 1.0f - fy) * (cx ? fx : 1.0f - fx);
            // a corner beyond the box can only carry weight 0 (a position rounded up to the box's last plane)
            if (w != 0.0f && bt + ct < kBoBox && by + cy < kBoBox && bx + cx < kBoBox) {
                const int i = ((bt + ct) * kBoBox + by + cy) * kBoBox + bx + cx;
                g.box_ck[i] = fmaf(g.s_ck[p], w, g.box_ck[i]);
                g.box_cv[i] = fmaf(g.s_cv[p], w, g.box_cv[i]);
            }
        }
    }

    // ---- out: one plane of ck and one of cv, [head][box position][token]; the block's groups hold consecutive
    //      tokens, so the block writes together, a run of tokens per box position
    __shared__ long long group_at[kBoGroups];
    if (gl == 0) group_at[threadIdx.x / kBoLanes] = static_cast<long long>(m) * kBoBoxCells * pr.N + n;
    __syncthreads();
    const long long plane_elems = pr.N * pr.heads * kBoBoxCells;
    const BoGroup* groups = reinterpret_cast<const BoGroup*>(bo_raw);
    for (int i = threadIdx.x; i < kBoGroups * kBoBoxCells; i += kBoThreads) {
        const int gi = i % kBoGroups, cellno = i / kBoGroups;
        if (block_first + gi >= pr.items) continue;
        const long long at = group_at[gi] + cellno * pr.N;
        planes[at] = split_bf16_pair(groups[gi].box_ck[cellno]);
        planes[plane_elems + at] = split_bf16_pair(groups[gi].box_cv[cellno]);
    }
}

}  // namespace

bool bounded_offsets_backward_covers(const Problem& pr, bool bf16) {
    if (!bf16 || (pr.d != 128 && pr.d != 64) || pr.kt != 3 || pr.kh != 3 || pr.kw != 3) return false;
    if (pr.q_begin != 0 || pr.q_count != pr.N) return false;
    // what the tile kernels count in 32 bits: positions inside a coefficient plane, planes walked
    const long long tiles = static_cast<long long>((pr.W + 7) / 8) * ((pr.H + 3) / 4) * ((pr.T + 3) / 4) * pr.heads;
    return pr.N * pr.heads * kBoBoxCells < (1LL << 31) && tiles * 3 * 9 < (1LL << 31);
}

// Bytes of workspace of the three kernels: the tables, then the two coefficient planes.
size_t bounded_offsets_backward_bytes(const Problem& pr) {
    const size_t tables = (static_cast<size_t>(pr.items) * bounded_offsets_table_floats() * sizeof(float) + 255) & ~static_cast<size_t>(255);
    return tables + static_cast<size_t>(pr.items) * kBoBoxCells * 2 * sizeof(uint32_t);
}

bool try_bounded_offsets_backward(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                                  const void* dout, void* dq, void* dk, void* dv, float* doffsets, void* workspace,
                                  const int* gate, const Problem& pr, cudaStream_t stream, cudaError_t* err) {
    *err = cudaSuccess;
    if (!bounded_offsets_backward_covers(pr, true)) return false;
    const size_t table_bytes = (static_cast<size_t>(pr.items) * bounded_offsets_table_floats() * sizeof(float) + 255) & ~static_cast<size_t>(255);
    float* table = static_cast<float*>(workspace);
    uint32_t* planes = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + table_bytes);
    if (!try_bounded_offsets_tables(q, k, v, dout, table, pr, gate, stream, err)) return false;
    if (*err != cudaSuccess) return true;
    const size_t smem = sizeof(BoGroup) * kBoGroups;
    *err = cudaFuncSetAttribute(bounded_offsets_backward_query_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(smem));
    if (*err != cudaSuccess) return true;
    const long long blocks = (pr.items + kBoGroups - 1) / kBoGroups;
    bounded_offsets_backward_query_kernel<<<static_cast<unsigned>(blocks), kBoThreads, smem, stream>>>(
        offsets, lse, table, doffsets, planes, gate, pr);
    *err = cudaGetLastError();
    if (*err != cudaSuccess) return true;
    // the tables kernel ran, so the plane kernel's shape is covered too; should its launch be refused, the
    // caller gets the error rather than half a result
    if (!try_bounded_offsets_planes_grad(q, k, dout, reinterpret_cast<const float*>(planes), dq, dk, dv, pr, gate, stream, err))
        *err = cudaErrorInvalidValue;
    return true;
}

}  // namespace dsa3d
