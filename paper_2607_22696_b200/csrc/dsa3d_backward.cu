// Backward of 3D Deformable Slide Attention: dQ, dK, dV and dOffsets.
//
// Two kernels.
//
// backward_kernel (one group of LPR = d / VEC lanes per (token, head) item, head-major
// order, as in the forward).  The sampling weights are recomputed from the offsets, the
// softmax weights from the saved lse; nothing of size N*P*d exists.
//   Pass 1 (gather): for every sample the corner rows of K and V are loaded once; the lane
//   partials of  s = sum_c w_c (q.K_c),  g = sum_c w_c (dO.V_c)  and of the six
//   derivative sums  A_a = sum_c (dw_c/da)(q.K_c),  B_a = sum_c (dw_c/da)(dO.V_c)  are
//   reduced over the group; alpha_p = exp(s_p - lse).  With delta = sum_p alpha_p g_p,
//   dQ = scale * (sum_p alpha_p g_p k_p - delta * sum_p alpha_p k_p) needs no second look
//   at K.  The eight per-sample numbers are parked in shared memory.
//   Pass 2: dS_p = alpha_p (g_p - delta);  dOffsets[p, a] = scale dS_p A_a + alpha_p B_a.
//   The two scatter coefficients of the sample, ck_p = scale dS_p and cv_p = alpha_p, are
//   written out for the tile kernel; corners that fall OUTSIDE the halo box of the query's
//   tile are scattered right here, dK[corner] += w_c ck_p q and dV[corner] += w_c cv_p dO,
//   with 16-byte vector reductions (red.global.add.v4.f32) into fp32 accumulators.
//
// scatter_tile_kernel (bf16 storage; one CTA per (head, tile of TQ queries), persistent).
//   The dK/dV contributions of a tile of neighbouring queries land on a few thousand key
//   rows around the tile, ~10 contributions per row.  Sending each one to L2 as a 512-byte
//   fp32 reduction is what bounds the simple scheme (L2 reduction throughput), so the tile
//   kernel sums them on chip first: it bins the (query, sample, corner) contributions of
//   the tile by target row (counting sort, counters in shared memory, 16-byte entries
//   {row offset, fp32 coefficient pair} in a per-CTA global scratch), then each group of
//   d/8 lanes (a half-warp at 128 channels, a quarter-warp at 64) owns a row, walks its entries, accumulates  coefficient x q-row  and  coefficient x
//   dO-row  in fp32 registers from the tile's q/dO rows held in shared memory, and issues
//   ONE reduction per row and tensor.
#include <type_traits>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"

namespace dsa3d {

constexpr int kStats = 8;   // per sample: alpha, g, A_t, A_y, A_x, B_t, B_y, B_x

#ifndef DSA3D_BWD_MINBLOCKS
#define DSA3D_BWD_MINBLOCKS 3
#endif

// The 128-channel bf16 kernel (two 16-byte vectors per lane, 128 registers): blocks of 128 threads, four
// per SM - the same 16 warps as two blocks of 256, in finer pieces (3 % faster).
#ifndef DSA3D_BWD_THREADS_NV2
#define DSA3D_BWD_THREADS_NV2 128
#endif
#ifndef DSA3D_BWD_MINBLOCKS_NV2
#define DSA3D_BWD_MINBLOCKS_NV2 4
#endif

template <typename T, int D, int NV>
__global__ void __launch_bounds__(NV == 2 ? DSA3D_BWD_THREADS_NV2 : 256, NV == 2 ? DSA3D_BWD_MINBLOCKS_NV2 : DSA3D_BWD_MINBLOCKS)
backward_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                const float* __restrict__ offsets, const float* __restrict__ lse,
                const T* __restrict__ dout, T* __restrict__ dq, float* __restrict__ acc_dk,
                float* __restrict__ acc_dv, float* __restrict__ doffsets, float2* __restrict__ coef,
                const Problem pr) {
    using E = Elt<T, NV>;
    using Row = typename E::Row;
    constexpr int VEC = E::VEC;
    constexpr int LPR = D / VEC;
    extern __shared__ float smem[];
    if (gated_off(pr)) return;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (LPR - 1);
    constexpr unsigned gmask = kFullMask;
    long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    const long long warp_first = (static_cast<long long>(blockIdx.x) * blockDim.x + (threadIdx.x & ~31)) / LPR;
    if (warp_first >= pr.items) return;                  // whole warp past the end
    const bool active = item < pr.items;                 // a trailing group repeats the last item, stores off
    if (!active) item = pr.items - 1;
    float* stats = smem + static_cast<size_t>(threadIdx.x / LPR) * pr.P * kStats;   // [P][8] of this group

    const int m = static_cast<int>(item / pr.q_count);
    const long long n = pr.q_begin + (item - static_cast<long long>(m) * pr.q_count);
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const long long row = n * pr.heads + m;
    const int ch = gl * VEC;
    const float scale = rsqrtf(static_cast<float>(D));
    const long long tok_stride = static_cast<long long>(pr.heads) * D;
    const long long sx = tok_stride;
    const long long sy = static_cast<long long>(pr.W) * sx;      // 64-bit once, so that the pointer
    const long long st = static_cast<long long>(pr.H) * sy;      // arithmetic below needs no widening

    const Row qr = E::load(q + row * D + ch);
    const Row dor = E::load(dout + row * D + ch);
    const float lse2 = __ldg(lse + row) * kLog2e;            // lse in log2 units
    const float* off_row = offsets + row * pr.P * 3;
    const long long head_off = static_cast<long long>(m) * D + ch;
    const T* kh = k + head_off;
    const long long v_minus_k = v - k;                       // same layout: V row = K row + this
    [[maybe_unused]] const long long kv_extent = pr.N * pr.heads * D;      // elements of K, V, dK, dV: checked build

    float u_acc[VEC], kbar[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) u_acc[e] = kbar[e] = 0.0f;
    float delta = 0.0f;

    // ---------------------------------------------------------------- pass 1: gather
    // Integer-offset regime: when every sample of every item of this warp sits exactly on a grid position
    // (one look at the offsets decides), a sample's value needs corner (0,0,0) alone and its one-sided
    // derivatives the +1 neighbour along each axis: four rows of K and of V, loaded back to back, instead
    // of eight.  The two regimes are two instances of the same loop, so that neither pays for the other's
    // registers.
    bool warp_on_lattice = true;
    for (int p = gl; p < pr.P; p += LPR) {
        const float* o3 = off_row + p * 3;
        const float ot = __ldg(o3), oy = __ldg(o3 + 1), ox = __ldg(o3 + 2);
        warp_on_lattice = warp_on_lattice && ot == floorf(ot) && oy == floorf(oy) && ox == floorf(ox);
    }
    warp_on_lattice = __all_sync(kFullMask, warp_on_lattice);
    auto pass1 = [&](auto lattice_tag) {
        constexpr bool lattice_chunk = decltype(lattice_tag)::value;
        for (int pb = 0; pb < pr.P; pb += LPR) {
            Sample mine;
            mine.base = 0; mine.mask = 0u; mine.ft = mine.fy = mine.fx = 0.0f;
            if (pb + gl < pr.P) mine = to_sample(pr, make_cell(pr, t, y, x, pb + gl, off_row + (pb + gl) * 3));
            const int cnt = min(LPR, pr.P - pb);
            for (int j = 0; j < cnt; ++j) {
                const Sample s = group_bcast<LPR>(mine, j, gmask);
                const float wt[2] = {1.0f - s.ft, s.ft}, wy[2] = {1.0f - s.fy, s.fy}, wx[2] = {1.0f - s.fx, s.fx};
                const T* kp4[4];             // corner row pointers per (ct, cy); cx = 1 is one token further
                kp4[0] = kh + s.base * tok_stride;
                kp4[1] = kp4[0] + sy;
                kp4[2] = kp4[0] + st;
                kp4[3] = kp4[2] + sy;
                float w[8];
                {
                    const float wty[4] = {wt[0] * wy[0], wt[0] * wy[1], wt[1] * wy[0], wt[1] * wy[1]};
    #pragma unroll
                    for (int c = 0; c < 8; ++c) w[c] = wty[c >> 1] * wx[c & 1];
                }
                float a[8], b[8];            // lane partials of q.K_c and dO.V_c (0 for corners not loaded)
                float kp[VEC];
    #pragma unroll
                for (int e = 0; e < VEC; ++e) kp[e] = 0.0f;
                const bool full = !lattice_chunk && s.mask == 0xffu && s.ft != 0.0f && s.fy != 0.0f && s.fx != 0.0f;
                if (full) {                    // every corner inside the grid and needed: 16 loads back to back
                    Row kk[8], vv[8];
    #pragma unroll
                    for (int c = 0; c < 8; ++c) kk[c] = E::load(kp4[c >> 1] + (c & 1) * sx);
    #pragma unroll
                    for (int c = 0; c < 8; ++c) vv[c] = E::load(kp4[c >> 1] + (c & 1) * sx + v_minus_k);
    #pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        a[c] = E::dot(qr, kk[c], 0.0f);
                        b[c] = E::dot(dor, vv[c], 0.0f);
                        E::axpy(w[c], kk[c], kp);
                    }
                } else if (lattice_chunk) {
                    // corners 0, 1 (x+1), 2 (y+1), 4 (t+1)
                    Row k0 = E::zero(), k1 = E::zero(), k2 = E::zero(), k4 = E::zero();
                    Row v0 = E::zero(), v1 = E::zero(), v2 = E::zero(), v4 = E::zero();
                    if ((s.mask & 1u) && DSA3D_IN_RANGE(pr, kp4[0] - k, kv_extent, 5)) { k0 = E::load(kp4[0]); v0 = E::load(kp4[0] + v_minus_k); }
                    if ((s.mask & 2u) && DSA3D_IN_RANGE(pr, kp4[0] + sx - k, kv_extent, 5)) { k1 = E::load(kp4[0] + sx); v1 = E::load(kp4[0] + sx + v_minus_k); }
                    if ((s.mask & 4u) && DSA3D_IN_RANGE(pr, kp4[1] - k, kv_extent, 5)) { k2 = E::load(kp4[1]); v2 = E::load(kp4[1] + v_minus_k); }
                    if ((s.mask & 16u) && DSA3D_IN_RANGE(pr, kp4[2] - k, kv_extent, 5)) { k4 = E::load(kp4[2]); v4 = E::load(kp4[2] + v_minus_k); }
                    a[0] = E::dot(qr, k0, 0.0f); b[0] = E::dot(dor, v0, 0.0f);
                    a[1] = E::dot(qr, k1, 0.0f); b[1] = E::dot(dor, v1, 0.0f);
                    a[2] = E::dot(qr, k2, 0.0f); b[2] = E::dot(dor, v2, 0.0f);
                    a[4] = E::dot(qr, k4, 0.0f); b[4] = E::dot(dor, v4, 0.0f);
                    a[3] = b[3] = a[5] = b[5] = a[6] = b[6] = a[7] = b[7] = 0.0f;
                    E::to_float(k0, kp);                                  // weight 1 on corner (0,0,0), 0 on the others
                } else {
    #pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int ct = c >> 2, cy = (c >> 1) & 1, cx = c & 1;
                        // a corner matters if its weight or one of its weight derivatives is non-zero
                        const bool needed = (w[c] != 0.0f) | (wy[cy] * wx[cx] != 0.0f) | (wt[ct] * wx[cx] != 0.0f) |
                                            (wt[ct] * wy[cy] != 0.0f);
                        a[c] = b[c] = 0.0f;
                        if (((s.mask >> c) & 1u) && needed && DSA3D_IN_RANGE(pr, kp4[c >> 1] + cx * sx - k, kv_extent, 6)) {
                            const T* pk = kp4[c >> 1] + cx * sx;
                            const Row kk = E::load(pk);
                            const Row vv = E::load(pk + v_minus_k);
                            a[c] = E::dot(qr, kk, 0.0f);
                            b[c] = E::dot(dor, vv, 0.0f);
                            E::axpy(w[c], kk, kp);
                        }
                    }
                }
                // r = (s, g, A_t, A_y, A_x, B_t, B_y, B_x) as lane partials, then summed over the group
                float r[kStats];
                trilerp_grad(a, s.ft, s.fy, s.fx, r[0], r[2], r[3], r[4]);
                trilerp_grad(b, s.ft, s.fy, s.fx, r[1], r[5], r[6], r[7]);
                float sdot, g;
                if constexpr (LPR >= 8) {
                    group_reduce8<LPR>(r, gl, gmask);
                    sdot = __shfl_sync(gmask, r[0], reduce8_lane<LPR>(0), LPR);
                    g = __shfl_sync(gmask, r[0], reduce8_lane<LPR>(1), LPR);
                } else {
    #pragma unroll
                    for (int i = 0; i < kStats; ++i) r[i] = group_sum<LPR>(r[i], gmask);
                    sdot = r[0];
                    g = r[1];
                }
                const float alpha = exp2f(fmaf(sdot, scale * kLog2e, -lse2));
                const float ag = alpha * g;
                delta += ag;
                if constexpr (NV == 2) {
    #pragma unroll
                    for (int e = 0; e < VEC; e += 2) {
                        fma2(u_acc[e], u_acc[e + 1], ag, ag, kp[e], kp[e + 1]);
                        fma2(kbar[e], kbar[e + 1], alpha, alpha, kp[e], kp[e + 1]);
                    }
                } else {
    #pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        u_acc[e] = fmaf(ag, kp[e], u_acc[e]);
                        kbar[e] = fmaf(alpha, kp[e], kbar[e]);
                    }
                }
                float* sts = stats + (pb + j) * kStats;
                if constexpr (LPR >= 8) {
                    const int idx = reduce8_index<LPR>(gl);
                    if (gl == reduce8_lane<LPR>(idx)) sts[idx] = idx == 0 ? alpha : r[0];   // slot 1 keeps g
                } else if (gl == 0) {
                    sts[0] = alpha; sts[1] = g;
    #pragma unroll
                    for (int i = 2; i < kStats; ++i) sts[i] = r[i];
                }
            }
        }
    };
    if (warp_on_lattice) pass1(std::true_type{});
    else pass1(std::false_type{});
    {
        float dqv[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) dqv[e] = scale * fmaf(-delta, kbar[e], u_acc[e]);
        if (active) E::store(dq + row * D + ch, dqv);
    }
    __syncwarp();

    // ------------------------------------------- pass 2: dOffsets, coefficients, far scatter
    float qf[VEC], dof[VEC];
    E::to_float(qr, qf);
    E::to_float(dor, dof);
    float* dk_h = acc_dk + head_off;
    float* dv_h = acc_dv + head_off;
    float* doff_row = doffsets + row * pr.P * 3;
    for (int pb = 0; pb < pr.P; pb += LPR) {
        Sample mine;
        mine.base = 0; mine.mask = 0u; mine.ft = mine.fy = mine.fx = 0.0f;
        float my_ck = 0.0f, my_cv = 0.0f;
        if (pb + gl < pr.P) {
            const int p = pb + gl;
            const Cell cell = make_cell(pr, t, y, x, p, off_row + p * 3);
            mine = to_sample(pr, cell);
            // corners the tile kernel (or the key-block kernel) does not take
            if (pr.key_blocks) mine.mask = active ? block_lists_append(pr, cell, t, y, x, m, p) : 0u;
            else mine.mask = cell.mask & ~halo_corner_mask(pr, cell, t, y, x);
            if (!active) mine.mask = 0u;
            const float* sts = stats + p * kStats;
            const float alpha = sts[0];
            const float dS = alpha * (sts[1] - delta);
            my_ck = scale * dS;
            my_cv = alpha;
            if (active) {
                doff_row[p * 3 + 0] = fmaf(my_ck, sts[2], alpha * sts[5]);
                doff_row[p * 3 + 1] = fmaf(my_ck, sts[3], alpha * sts[6]);
                doff_row[p * 3 + 2] = fmaf(my_ck, sts[4], alpha * sts[7]);
                if (coef) coef[row * pr.P + p] = make_float2(my_ck, my_cv);
            }
        }
        const int cnt = min(LPR, pr.P - pb);
        for (int j = 0; j < cnt; ++j) {
            const unsigned mask = __shfl_sync(gmask, mine.mask, j, LPR);
            if (!__any_sync(kFullMask, mask != 0u)) continue;      // warp-uniform: shuffles follow
            const Sample s = group_bcast<LPR>(mine, j, gmask);
            const float ck = __shfl_sync(gmask, my_ck, j, LPR);
            const float cv = __shfl_sync(gmask, my_cv, j, LPR);
            const float wt[2] = {1.0f - s.ft, s.ft}, wy[2] = {1.0f - s.fy, s.fy}, wx[2] = {1.0f - s.fx, s.fx};
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float w = wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1];
                if (((s.mask >> c) & 1u) && w != 0.0f &&
                    DSA3D_IN_RANGE(pr, head_off + s.base * tok_stride + ((c >> 2) * st + ((c >> 1) & 1) * sy + (c & 1) * sx), kv_extent, 7)) {
                    const long long o = s.base * tok_stride + ((c >> 2) * st + ((c >> 1) & 1) * sy + (c & 1) * sx);
                    const float wk = w * ck, wv = w * cv;
                    float* pk = dk_h + o;
                    float* pv = dv_h + o;
#pragma unroll
                    for (int e = 0; e < VEC; e += 4) {
                        red_add_v4(pk + e, wk * qf[e], wk * qf[e + 1], wk * qf[e + 2], wk * qf[e + 3]);
                        red_add_v4(pv + e, wv * dof[e], wv * dof[e + 1], wv * dof[e + 2], wv * dof[e + 3]);
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Tile scatter (bf16 storage).
// ---------------------------------------------------------------------------------------
#ifndef DSA3D_TILE_THREADS
#define DSA3D_TILE_THREADS 1024
#endif
constexpr int kTileThreads = DSA3D_TILE_THREADS;

template <int D>
__global__ void __launch_bounds__(kTileThreads, 1)
scatter_tile_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ dout,
                    const float* __restrict__ offsets, const float2* __restrict__ coef,
                    float* __restrict__ acc_dk, float* __restrict__ acc_dv, TileEntry* __restrict__ scratch,
                    const long long scratch_entries_per_cta, const Problem pr) {
    constexpr int VPR = D / 8;                       // 16-byte vectors per row
    constexpr int kPairBytes = 2 * VPR * 16;         // one query's q row followed by its dO row
    constexpr unsigned kFull = 0xffffffffu;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (gated_off(pr)) return;
    const int TQ = pr.tile_t * pr.tile_y * pr.tile_x;
    const int et = pr.tile_t + 2 * pr.halo, ey = pr.tile_y + 2 * pr.halo, ex = pr.tile_x + 2 * pr.halo;
    const int NB = et * ey * ex;
    uint4* rows = reinterpret_cast<uint4*>(smem_raw);                                   // [TQ][2][VPR]
    unsigned* cursor = reinterpret_cast<unsigned*>(smem_raw + static_cast<size_t>(TQ) * kPairBytes);   // [NB]
    __shared__ unsigned warp_sums[kTileThreads / 32];
    __shared__ uint4 ent_stage[kTileThreads];          // one entry per lane, read back by every lane of its group

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kTileThreads / 32;
    const int tiles_per_head = pr.tt_count * pr.tiles_y * pr.tiles_x;
    const long long total_tiles = static_cast<long long>(tiles_per_head) * pr.heads;
    TileEntry* my_scratch = scratch + static_cast<long long>(blockIdx.x) * scratch_entries_per_cta;
    const long long tok_stride = static_cast<long long>(pr.heads) * D;

    for (long long tile_id = blockIdx.x; tile_id < total_tiles; tile_id += gridDim.x) {
        const int m = static_cast<int>(tile_id / tiles_per_head);
        int rem = static_cast<int>(tile_id - static_cast<long long>(m) * tiles_per_head);
        const int tx = rem % pr.tiles_x; rem /= pr.tiles_x;
        const int ty = rem % pr.tiles_y;
        const int tt = pr.tt_begin + rem / pr.tiles_y;
        const int t0 = tt * pr.tile_t, y0 = ty * pr.tile_y, x0 = tx * pr.tile_x;
        const int lo_t = t0 - pr.halo, lo_y = y0 - pr.halo, lo_x = x0 - pr.halo;

        // ---- stage the tile's q and dO rows, clear the bin counters
        for (int i = tid; i < NB; i += kTileThreads) cursor[i] = 0u;
        for (int i = tid; i < TQ * VPR; i += kTileThreads) {
            const int ql = i / VPR, vec = i - ql * VPR;
            const int lx = ql % pr.tile_x, ly = (ql / pr.tile_x) % pr.tile_y, lt = ql / (pr.tile_x * pr.tile_y);
            const int t = t0 + lt, y = y0 + ly, x = x0 + lx;
            uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
            if (t < pr.T && y < pr.H && x < pr.W) {
                const long long n = (static_cast<long long>(t) * pr.H + y) * pr.W + x;
                const long long o = (n * pr.heads + m) * D + vec * 8;
                a = __ldg(reinterpret_cast<const uint4*>(q + o));
                b = __ldg(reinterpret_cast<const uint4*>(dout + o));
            }
            rows[ql * 2 * VPR + vec] = a;
            rows[ql * 2 * VPR + VPR + vec] = b;
        }
        __syncthreads();

        // ---- count and fill: two sweeps over the (query, sample) pairs of the tile; a warp
        //      takes one query at a time, its lanes the samples
        for (int sweep = 0; sweep < 2; ++sweep) {
            for (int ql = warp; ql < TQ; ql += kWarps) {
                const int lx = ql % pr.tile_x, ly = (ql / pr.tile_x) % pr.tile_y, lt = ql / (pr.tile_x * pr.tile_y);
                const int t = t0 + lt, y = y0 + ly, x = x0 + lx;
                if (t >= pr.T || y >= pr.H || x >= pr.W) continue;
                const long long n = (static_cast<long long>(t) * pr.H + y) * pr.W + x;
                const long long row = n * pr.heads + m;
                for (int p = lane; p < pr.P; p += 32) {
                    const Cell cell = make_cell(pr, t, y, x, p, offsets + (row * pr.P + p) * 3);
                    const unsigned mask =
                        cell.mask & corner_mask(cell.it - lo_t, cell.iy - lo_y, cell.ix - lo_x, et, ey, ex);
                    if (mask == 0u) continue;
                    const float wt[2] = {1.0f - cell.ft, cell.ft}, wy[2] = {1.0f - cell.fy, cell.fy},
                                wx[2] = {1.0f - cell.fx, cell.fx};
                    const int bin0 = ((cell.it - lo_t) * ey + (cell.iy - lo_y)) * ex + (cell.ix - lo_x);
                    float2 cf = make_float2(0.f, 0.f);
                    if (sweep == 1) cf = __ldg(coef + row * pr.P + p);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float w = wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1];
                        if (((mask >> c) & 1u) && w != 0.0f) {
                            const int bin = bin0 + ((c >> 2) * ey + ((c >> 1) & 1)) * ex + (c & 1);
                            if (!DSA3D_IN_RANGE(pr, bin, NB, 8)) continue;
                            const unsigned slot = atomicAdd(&cursor[bin], 1u);
                            if (sweep == 1 && DSA3D_IN_RANGE(pr, slot, scratch_entries_per_cta, 9)) {
                                my_scratch[slot] = make_uint4(static_cast<unsigned>(ql * kPairBytes),
                                                              __float_as_uint(w * cf.x), __float_as_uint(w * cf.y), 0u);
                            }
                        }
                    }
                }
            }
            __syncthreads();
            if (sweep == 0) {
                // exclusive prefix sum of the NB counters, in place
                const int per = (NB + kTileThreads - 1) / kTileThreads;
                const int b0 = tid * per, b1 = min(NB, b0 + per);
                unsigned local = 0;
                for (int i = b0; i < b1; ++i) local += cursor[i];
                unsigned incl = local;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned nb = __shfl_up_sync(kFull, incl, o);
                    if (lane >= o) incl += nb;
                }
                if (lane == 31) warp_sums[warp] = incl;
                __syncthreads();
                if (tid < 32) {
                    const unsigned ws = tid < kWarps ? warp_sums[tid] : 0u;
                    unsigned wi = ws;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned nb = __shfl_up_sync(kFull, wi, o);
                        if (tid >= o) wi += nb;
                    }
                    if (tid < kWarps) warp_sums[tid] = wi - ws;     // exclusive
                }
                __syncthreads();
                unsigned run = warp_sums[warp] + incl - local;
                for (int i = b0; i < b1; ++i) {
                    const unsigned c = cursor[i];
                    cursor[i] = run;
                    run += c;
                }
                __syncthreads();
            }
        }
        // after the fill sweep cursor[b] is the END of bin b; its start is the end of bin b-1

        // ---- reduce: a row is VPR 16-byte vectors, one per lane, so a warp takes 32 / VPR
        //      neighbouring key rows at once (two at 128 channels); every group runs the same
        //      number of steps (the shorter lists are padded with zero entries)
        {
            constexpr int GW = VPR;                          // lanes per key row
            constexpr int kGroups = 32 / GW;
            const int grp = lane / GW, hl = lane & (GW - 1);
            [[maybe_unused]] const int lane0 = lane & ~(GW - 1);              // first lane of this group
            const unsigned char* my_rows = smem_raw + hl * 16;
            for (int firstbin = warp * kGroups; firstbin < NB; firstbin += kWarps * kGroups) {
                const int bin = firstbin + grp;
                unsigned start = 0u, end = 0u;
                if (bin < NB) {
                    end = cursor[bin];
                    start = bin == 0 ? 0u : cursor[bin - 1];
                }
                const unsigned cnt_mine = end - start;
                unsigned cnt_max = cnt_mine;
#pragma unroll
                for (int o = GW; o < 32; o <<= 1) cnt_max = max(cnt_max, __shfl_xor_sync(kFull, cnt_max, o));
                if (cnt_max == 0u) continue;
                float ak[8], av[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) ak[e] = av[e] = 0.0f;
                for (unsigned base = 0; base < cnt_max; base += GW) {
                    uint4 ent = make_uint4(0u, 0u, 0u, 0u);               // offset 0, coefficients 0
                    if (base + hl < cnt_mine) ent = __ldcg(my_scratch + start + base + hl);
                    const int steps = static_cast<int>(min(static_cast<unsigned>(GW), cnt_max - base));
                    // the group's entries go through shared memory: one broadcast read per step
                    // instead of three shuffles
                    __syncwarp();
                    ent_stage[tid] = ent;
                    __syncwarp();
                    const uint4* grp_ent = ent_stage + (tid & ~(GW - 1));
#pragma unroll 4
                    for (int j = 0; j < steps; ++j) {
                        const uint4 ej = grp_ent[j];
                        const unsigned off = ej.x;
                        const float ck = __uint_as_float(ej.y), cv = __uint_as_float(ej.z);
                        const uint4 a = *reinterpret_cast<const uint4*>(my_rows + off);
                        const uint4 b = *reinterpret_cast<const uint4*>(my_rows + off + VPR * 16);
                        const unsigned aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
                        // two fp32 FMAs per instruction (fma.rn.f32x2): same arithmetic, fewer issue slots
                        unsigned long long ckk, cvv;
                        asm("mov.b64 %0, {%1, %1};" : "=l"(ckk) : "f"(ck));
                        asm("mov.b64 %0, {%1, %1};" : "=l"(cvv) : "f"(cv));
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            unsigned long long xa, xb, pa, pb;
                            asm("mov.b64 %0, {%1, %2};" : "=l"(xa) : "r"(aw[i] << 16), "r"(aw[i] & 0xffff0000u));
                            asm("mov.b64 %0, {%1, %2};" : "=l"(xb) : "r"(bw[i] << 16), "r"(bw[i] & 0xffff0000u));
                            asm("mov.b64 %0, {%1, %2};" : "=l"(pa) : "f"(ak[2 * i]), "f"(ak[2 * i + 1]));
                            asm("mov.b64 %0, {%1, %2};" : "=l"(pb) : "f"(av[2 * i]), "f"(av[2 * i + 1]));
                            asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(pa) : "l"(ckk), "l"(xa));
                            asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(pb) : "l"(cvv), "l"(xb));
                            asm("mov.b64 {%0, %1}, %2;" : "=f"(ak[2 * i]), "=f"(ak[2 * i + 1]) : "l"(pa));
                            asm("mov.b64 {%0, %1}, %2;" : "=f"(av[2 * i]), "=f"(av[2 * i + 1]) : "l"(pb));
                        }
                    }
                }
                if (cnt_mine > 0u) {
                    const int bx = bin % ex, by = (bin / ex) % ey, bt = bin / (ex * ey);
                    const long long tok = (static_cast<long long>(lo_t + bt) * pr.H + (lo_y + by)) * pr.W + (lo_x + bx);
                    const long long o = tok * tok_stride + static_cast<long long>(m) * D + hl * 8;
                    if (DSA3D_IN_RANGE(pr, tok, pr.N, 10)) {
                    red_add_v4(acc_dk + o, ak[0], ak[1], ak[2], ak[3]);
                    red_add_v4(acc_dk + o + 4, ak[4], ak[5], ak[6], ak[7]);
                    red_add_v4(acc_dv + o, av[0], av[1], av[2], av[3]);
                    red_add_v4(acc_dv + o + 4, av[4], av[5], av[6], av[7]);
                    }
                }
            }
        }
        __syncthreads();     // the next tile reuses the rows, the counters and the scratch
    }
}

size_t tile_smem_bytes(const Problem& pr) {
    const size_t TQ = static_cast<size_t>(pr.tile_t) * pr.tile_y * pr.tile_x;
    const size_t NB = static_cast<size_t>(pr.tile_t + 2 * pr.halo) * (pr.tile_y + 2 * pr.halo) *
                      (pr.tile_x + 2 * pr.halo);
    return TQ * pr.d * 2 * 2 + NB * sizeof(unsigned);
}

// 16-byte vectors per lane: two for 128-channel bf16 rows (8 lanes per item, 4 items per warp,
// 2 blocks per SM), which halves the per-item bookkeeping of the backward; one otherwise.
#ifndef DSA3D_BWD_BF16_NV
#define DSA3D_BWD_BF16_NV 2
#endif
template <typename T, int D> struct BwdLaneWidth { static constexpr int NV = 1; };
template <> struct BwdLaneWidth<__nv_bfloat16, 128> { static constexpr int NV = DSA3D_BWD_BF16_NV; };

template <typename T, int D>
static cudaError_t launch_backward_t(const void* q, const void* k, const void* v, const float* offsets,
                                     const float* lse, const void* dout, void* dq, float* acc_dk,
                                     float* acc_dv, float* doffsets, float2* coef, const Problem& pr,
                                     cudaStream_t stream) {
    constexpr int NV = BwdLaneWidth<T, D>::NV;
    constexpr int LPR = D / Elt<T, NV>::VEC;
    // Shared memory holds 8 floats per (group, sample); shrink the block for large windows.
    int threads = NV == 2 ? DSA3D_BWD_THREADS_NV2 : 256;
    while (threads > 32 && static_cast<size_t>(threads / LPR) * pr.P * kStats * sizeof(float) > 64 * 1024)
        threads /= 2;
    const size_t smem = static_cast<size_t>(threads / LPR) * pr.P * kStats * sizeof(float);
    auto kern = backward_kernel<T, D, NV>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    if (NV == 2 && smem * DSA3D_BWD_MINBLOCKS_NV2 <= 56 * 1024) {
        // the per-sample statistics of the resident blocks fit a quarter of the SM's shared memory: ask for
        // that split, the rest of the array serves the corner gathers as L1
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 25);
        if (e != cudaSuccess) return e;
    }
    const long long groups_per_block = threads / LPR;
    const long long blocks = (pr.items + groups_per_block - 1) / groups_per_block;
    kern<<<static_cast<unsigned>(blocks), threads, smem, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), offsets, lse,
        static_cast<const T*>(dout), static_cast<T*>(dq), acc_dk, acc_dv, doffsets, coef, pr);
    return cudaGetLastError();
}

cudaError_t launch_backward(const void* q, const void* k, const void* v, const float* offsets,
                            const float* lse, const void* dout, void* dq, float* acc_dk, float* acc_dv,
                            float* doffsets, float2* coef, const Problem& pr, bool bf16,
                            cudaStream_t stream) {
#define DSA3D_CASE(DD)                                                                                   \
    case DD:                                                                                             \
        return bf16 ? launch_backward_t<__nv_bfloat16, DD>(q, k, v, offsets, lse, dout, dq, acc_dk,     \
                                                           acc_dv, doffsets, coef, pr, stream)           \
                    : launch_backward_t<float, DD>(q, k, v, offsets, lse, dout, dq, acc_dk, acc_dv,      \
                                                   doffsets, coef, pr, stream);
    switch (pr.d) {
        DSA3D_CASE(32)
        DSA3D_CASE(64)
        DSA3D_CASE(128)
    }
#undef DSA3D_CASE
    return cudaErrorInvalidValue;
}

template <int D>
static cudaError_t launch_scatter_tiles_t(const void* q, const void* dout, const float* offsets,
                                          const float2* coef, float* acc_dk, float* acc_dv, void* scratch,
                                          int ctas, long long entries_per_cta, const Problem& pr,
                                          cudaStream_t stream) {
    auto kern = scatter_tile_kernel<D>;
    const size_t smem = tile_smem_bytes(pr);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    const long long total_tiles = static_cast<long long>(pr.tt_count) * pr.tiles_y * pr.tiles_x * pr.heads;
    const int grid = static_cast<int>(total_tiles < ctas ? total_tiles : ctas);
    kern<<<grid, kTileThreads, smem, stream>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(dout), offsets, coef, acc_dk,
        acc_dv, static_cast<TileEntry*>(scratch), entries_per_cta, pr);
    return cudaGetLastError();
}

cudaError_t launch_scatter_tiles(const void* q, const void* dout, const float* offsets, const float2* coef,
                                 float* acc_dk, float* acc_dv, void* scratch, int ctas,
                                 long long entries_per_cta, const Problem& pr, cudaStream_t stream) {
    switch (pr.d) {
        case 32: return launch_scatter_tiles_t<32>(q, dout, offsets, coef, acc_dk, acc_dv, scratch, ctas, entries_per_cta, pr, stream);
        case 64: return launch_scatter_tiles_t<64>(q, dout, offsets, coef, acc_dk, acc_dv, scratch, ctas, entries_per_cta, pr, stream);
        case 128: return launch_scatter_tiles_t<128>(q, dout, offsets, coef, acc_dk, acc_dv, scratch, ctas, entries_per_cta, pr, stream);
    }
    return cudaErrorInvalidValue;
}

__global__ void __launch_bounds__(256)
convert_bf16_kernel(const float4* __restrict__ acc, uint2* __restrict__ dst, long long count4, const int* __restrict__ gate) {
    if (gate != nullptr && *gate == 0) return;      // the tile kernels of a bounded-offsets backward wrote dk and dv
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < count4; i += stride) {
        const float4 a = acc[i];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(a.z, a.w);
        dst[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
}

// Zeroes `count4` 16-byte pieces unless *gate is 0 (a gated backward whose tile kernels took the call needs
// no accumulators; an unconditional memset would cost it their size in HBM writes).
__global__ void __launch_bounds__(256)
gated_clear_kernel(uint4* __restrict__ dst, long long count4, const int* __restrict__ gate) {
    if (*gate == 0) return;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < count4; i += stride)
        dst[i] = make_uint4(0u, 0u, 0u, 0u);
}

cudaError_t launch_gated_clear(void* dst, size_t bytes, const int* gate, cudaStream_t stream) {
    const long long count4 = static_cast<long long>(bytes / 16);     // the accumulators are whole rows of d floats
    long long blocks = (count4 + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    if (blocks < 1) blocks = 1;
    gated_clear_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(static_cast<uint4*>(dst), count4, gate);
    return cudaGetLastError();
}

cudaError_t launch_convert_bf16(const float* acc, void* dst, long long count, cudaStream_t stream, const int* gate) {
    const long long count4 = count / 4;      // d is a multiple of 32, so count is a multiple of 4
    long long blocks = (count4 + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    if (blocks < 1) blocks = 1;
    convert_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(acc), reinterpret_cast<uint2*>(dst), count4, gate);
    return cudaGetLastError();
}

}  // namespace dsa3d
