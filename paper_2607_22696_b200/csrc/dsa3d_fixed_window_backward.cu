// Backward of the fixed-window variant (all offsets zero).  Every sample sits exactly on the
// grid position query + b(p), so nothing is interpolated and nothing needs an atomic:
//
//   fixed_window_backward_query_kernel   one group of lanes per (query, head).  The dot products
//       a = q.K_j and b = dO.V_j are taken once for every position j of the box the window and
//       its +1 neighbours span ((kt+1)(kh+1)(kw+1) positions, 54 of them used for 3x3x3; only
//       the window itself when dOffsets is not wanted), eight positions per transposed
//       reduction, into a small table in shared memory.  From the table: alpha_p, g_p, delta,
//       dS_p; dOffsets by the one-sided derivative of the trilinear weights at an integer
//       position, dDelta_a = score(j + e_a) - score(j) with score = scale dS_p a + alpha_p b
//       and positions outside the grid counting 0; the two coefficients scale dS_p and
//       alpha_p of every sample go to the workspace; dQ = sum_p scale dS_p K_j in a second
//       visit of the window's K rows.
//   fixed_window_backward_key_kernel     one group per (key, head): with a fixed window the
//       contributions to dK_j and dV_j come from the P queries j - b(p), so they are gathered:
//       dK_j = sum_p coefK[j - b(p), p] q_{j - b(p)},  dV_j = sum_p coefV[j - b(p), p] dO_{j - b(p)},
//       and written once in the storage type - no fp32 accumulators, no atomics, bitwise
//       deterministic.
#include <cuda_bf16.h>

#include <type_traits>

#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"

namespace dsa3d {
namespace {

// An fp32 value as two bf16 numbers whose sum is the value to 2^-17 relative: the nearest bf16 in the low
// half of the word, the nearest bf16 of what is left in the high half.
__device__ __forceinline__ uint32_t split_bf16_pair(float x) {
    const __nv_bfloat16 head = __float2bfloat16_rn(x);
    const __nv_bfloat16 rest = __float2bfloat16_rn(x - __bfloat162float(head));
    return static_cast<uint32_t>(__bfloat16_as_ushort(head)) | (static_cast<uint32_t>(__bfloat16_as_ushort(rest)) << 16);
}

// Resident blocks the table-fed kernel is compiled for (64 registers per thread at four; measured against
// three: backward 20.1 -> 19.5 ms for (3,7,7), 12.3 -> 11.9 for (3,5,5), 7.8 -> 7.6 for (3,3,3) on the sweep grid).
#ifndef DSA3D_FWB_TABLE_BLOCKS
#define DSA3D_FWB_TABLE_BLOCKS 4
#endif
// KT, KH, KW: the window when it is known at compile time (the shapes the table kernel covers: loop bounds,
// strides and the box layout then fold into the code), 0, 0, 0 = taken from the problem.
template <typename T, int D, bool TABLE, int KT = 0, int KH = 0, int KW = 0>
__global__ void __launch_bounds__(256, TABLE ? DSA3D_FWB_TABLE_BLOCKS : 1)
fixed_window_backward_query_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                   const float* __restrict__ lse, const T* __restrict__ dout, T* __restrict__ dq,
                                   float* __restrict__ doffsets, float2* __restrict__ coef,
                                   const float* __restrict__ table, const bool coef_planes, const Problem pr) {
    using E = Elt<T, 1>;
    using Row = typename E::Row;
    constexpr int VEC = E::VEC;
    constexpr int LPR = D / VEC;
    extern __shared__ float smem[];
    const int win_t = KT ? KT : pr.kt, win_y = KT ? KH : pr.kh, win_x = KT ? KW : pr.kw, n_samples = KT ? KT * KH * KW : pr.P;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (LPR - 1);
    constexpr unsigned gmask = kFullMask;
    long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    const long long warp_first = (static_cast<long long>(blockIdx.x) * blockDim.x + (threadIdx.x & ~31)) / LPR;
    const bool whole_warp_idle = warp_first >= pr.items;   // leaves after the block-wide table is built
    const bool active = item < pr.items;                 // a trailing group repeats the last item, stores off
    if (!active) item = pr.items - 1;

    const bool want_doff = doffsets != nullptr;
    // with a table the box always has the +1 neighbours (that is how the table is laid out)
    const bool wide = want_doff || TABLE;
    const int BT = win_t + (wide ? 1 : 0), BY = win_y + (wide ? 1 : 0), BX = win_x + (wide ? 1 : 0);
    const int NB = BT * BY * BX;
    const int NB8 = (NB + 7) & ~7;
    // per block: box_tab[NB8] = displacement of box position idx from the box origin and whether
    // it is used (a window cell, or the +1 neighbour of one along exactly one axis);
    // samp_tab[P] = box index of sample p's own position
    int4* box_tab = reinterpret_cast<int4*>(smem);
    int* samp_tab = reinterpret_cast<int*>(box_tab + NB8);
    float* group0 = reinterpret_cast<float*>(samp_tab + ((n_samples + 3) & ~3));
    for (int idx = threadIdx.x; idx < NB8; idx += blockDim.x) {
        const int bw = idx % BX, bv = (idx / BX) % BY, bu = idx / (BX * BY);
        const int far = (bu == win_t) + (bv == win_y) + (bw == win_x);
        box_tab[idx] = make_int4(bu, bv, bw, (idx < NB && far <= 1) ? 1 : 0);
    }
    for (int p = threadIdx.x; p < n_samples; p += blockDim.x) {
        const int w = p % win_x, vv = (p / win_x) % win_y, u = p / (win_x * win_y);
        samp_tab[p] = (u * BY + vv) * BX + w;
    }
    __syncthreads();
    if (whole_warp_idle) return;
    // per group: ta[NB8], tb[NB8] (dot products per box position), sa[P] (alpha), sk[P] (scale dS)
    float* ta = group0 + static_cast<size_t>(threadIdx.x / LPR) * (2 * NB8 + 2 * n_samples);
    float* tb = ta + NB8;
    float* sa = tb + NB8;
    float* sk = sa + n_samples;

    const int m = static_cast<int>(item / pr.q_count);
    const long long n = pr.q_begin + (item - static_cast<long long>(m) * pr.q_count);
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const long long row = n * pr.heads + m;
    const int ch = gl * VEC;
    const float scale = rsqrtf(static_cast<float>(D));
    const long long tok_stride = static_cast<long long>(pr.heads) * D;
    const T* kh = k + static_cast<long long>(m) * D + ch;
    const long long v_minus_k = v - k;
    const int ot = t - win_t / 2, oy = y - win_y / 2, ox = x - win_x / 2;      // box origin

    const float lse2 = __ldg(lse + row) * kLog2e;

    if constexpr (TABLE) {
        // ---- dot products from the table the tensor cores wrote: [item][a, b][NB8]
        const float* mine = table + row * (2 * NB8);
        for (int i = gl; i < NB8; i += LPR) {
            ta[i] = __ldg(mine + i);
            tb[i] = __ldg(mine + NB8 + i);
        }
    } else {
    const Row qr = E::load(q + row * D + ch);
    const Row dor = E::load(dout + row * D + ch);
    // ---- dot products over the box, eight positions per reduction: all 16 row loads of a chunk
    //      are issued before the first dot product
    for (int c8 = 0; c8 < NB8; c8 += 8) {
        Row kk[8], vv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int4 bt = box_tab[c8 + i];
            const int pt = ot + bt.x, py = oy + bt.y, px = ox + bt.z;
            const bool inside = bt.w && pt >= 0 && pt < pr.T && py >= 0 && py < pr.H && px >= 0 && px < pr.W;
            kk[i] = E::zero();
            vv[i] = E::zero();
            if (inside) {
                const T* pk = kh + ((static_cast<long long>(pt) * pr.H + py) * pr.W + px) * tok_stride;
                kk[i] = E::load(pk);
                vv[i] = E::load(pk + v_minus_k);
            }
        }
        float a8[8], b8[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            a8[i] = E::dot(qr, kk[i], 0.0f);
            b8[i] = E::dot(dor, vv[i], 0.0f);
        }
        if constexpr (LPR >= 8) {
            group_reduce8<LPR>(a8, gl, gmask);
            group_reduce8<LPR>(b8, gl, gmask);
            const int which = reduce8_index<LPR>(gl);
            if (gl == reduce8_lane<LPR>(which)) {
                ta[c8 + which] = a8[0];
                tb[c8 + which] = b8[0];
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                a8[i] = group_sum<LPR>(a8[i], gmask);
                b8[i] = group_sum<LPR>(b8[i], gmask);
            }
            if (gl == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i) { ta[c8 + i] = a8[i]; tb[c8 + i] = b8[i]; }
            }
        }
    }
    }
    __syncwarp();

    // ---- softmax weights, delta
    float delta = 0.0f;
    for (int p = gl; p < n_samples; p += LPR) {
        const int idx = samp_tab[p];
        const float alpha = exp2f(fmaf(ta[idx], scale * kLog2e, -lse2));     // a position outside the grid: logit 0
        sa[p] = alpha;
        delta = fmaf(alpha, tb[idx], delta);
    }
    delta = group_sum<LPR>(delta, gmask);

    // ---- dS, coefficients, dOffsets
    for (int p = gl; p < n_samples; p += LPR) {
        const int idx = samp_tab[p];
        const float alpha = sa[p];
        const float ck = scale * alpha * (tb[idx] - delta);
        sk[p] = ck;
        if (active) {
            if (!coef_planes) coef[row * n_samples + p] = make_float2(ck, alpha);
            if (want_doff) {
                const float s0 = fmaf(ck, ta[idx], alpha * tb[idx]);
                float* dst = doffsets + (row * n_samples + p) * 3;
                dst[0] = fmaf(ck, ta[idx + BY * BX], alpha * tb[idx + BY * BX]) - s0;
                dst[1] = fmaf(ck, ta[idx + BX], alpha * tb[idx + BX]) - s0;
                dst[2] = fmaf(ck, ta[idx + 1], alpha * tb[idx + 1]) - s0;
            }
        }
    }
    __syncwarp();

    if (coef_planes) {
        // For the plane-by-plane tile kernel the coefficients go out as one plane of ck and one of cv, each
        // [head][sample][token], so that the outputs of a tile row find the coefficients of one window cell
        // side by side - and already as that kernel multiplies them: a bf16 head and the bf16 remainder of
        // the fp32 value in one word (relative error of the pair 2^-17).  The block's groups hold consecutive tokens: the block writes together, a run of
        // tokens per sample, from the groups' arrays in shared memory.
        const int groups = blockDim.x / LPR;
        long long* group_at = reinterpret_cast<long long*>(group0 + static_cast<size_t>(groups) * (2 * NB8 + 2 * n_samples));
        if (gl == 0) group_at[threadIdx.x / LPR] = static_cast<long long>(m) * n_samples * pr.N + n;
        __syncthreads();                                   // warps with no item at all have left: they count as arrived
        uint32_t* planes = reinterpret_cast<uint32_t*>(coef);
        const long long plane_elems = pr.N * pr.heads * n_samples;
        const long long block_first = static_cast<long long>(blockIdx.x) * groups;     // item of group 0
        // the threads still here: the warps up to the last one that holds an item
        const long long lanes_with_items = (pr.items - block_first) * LPR;
        const int live = lanes_with_items >= blockDim.x ? static_cast<int>(blockDim.x) : static_cast<int>((lanes_with_items + 31) / 32 * 32);
        for (int i = threadIdx.x; i < groups * n_samples; i += live) {
            const int g = i % groups, p = i / groups;
            if (block_first + g >= pr.items) continue;     // a group without an item (its arrays and position are not set)
            const long long at = group_at[g];
            const float* ga = group0 + static_cast<size_t>(g) * (2 * NB8 + 2 * n_samples) + 2 * NB8;     // sa, then sk
            planes[at + p * pr.N] = split_bf16_pair(ga[n_samples + p]);
            planes[plane_elems + at + p * pr.N] = split_bf16_pair(ga[p]);
        }
    }

    // ---- dQ = sum_p (scale dS_p) K_j over the window cells inside the grid (unless the tile kernel forms it)
    if (dq == nullptr) return;
    float dqv[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) dqv[e] = 0.0f;
    for (int p0 = 0; p0 < n_samples; p0 += 8) {
        Row kk[8];
        float cks[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            kk[i] = E::zero();
            cks[i] = 0.0f;
            if (p0 + i < n_samples) {
                const int4 bt = box_tab[samp_tab[p0 + i]];
                const int pt = ot + bt.x, py = oy + bt.y, px = ox + bt.z;
                if (pt >= 0 && pt < pr.T && py >= 0 && py < pr.H && px >= 0 && px < pr.W) {
                    kk[i] = E::load(kh + ((static_cast<long long>(pt) * pr.H + py) * pr.W + px) * tok_stride);
                    cks[i] = sk[p0 + i];
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) E::axpy_paired(cks[i], kk[i], dqv);
    }
    if (active) E::store(dq + row * D + ch, dqv);
}

template <typename T, int D>
__global__ void __launch_bounds__(256)
fixed_window_backward_key_kernel(const T* __restrict__ q, const T* __restrict__ dout, const float2* __restrict__ coef,
                                 T* __restrict__ dk, T* __restrict__ dv, const Problem pr) {
    using E = Elt<T, 1>;
    using Row = typename E::Row;
    constexpr int VEC = E::VEC;
    constexpr int LPR = D / VEC;
    const int gl = threadIdx.x & (LPR - 1);
    const long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    if (item >= pr.items) return;
    const int m = static_cast<int>(item / pr.q_count);
    const long long n = item - static_cast<long long>(m) * pr.q_count;
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const int ch = gl * VEC;
    float ak[VEC], av[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) ak[e] = av[e] = 0.0f;
    // The query whose window cell p = (u, vv, w) is this key sits at key - b(p): walking w moves it one token
    // back, so the row and coefficient pointers are stepped instead of recomputed, and the range tests are
    // taken once per loop level.
    const long long tok = static_cast<long long>(pr.heads) * D;              // elements from one token to the next
    const long long coef_tok = static_cast<long long>(pr.heads) * pr.P;
    for (int u = 0; u < pr.kt; ++u) {
        const int qt = t - (u - pr.kt / 2);
        if (qt < 0 || qt >= pr.T) continue;
        for (int vv = 0; vv < pr.kh; ++vv) {
            const int qy = y - (vv - pr.kh / 2);
            if (qy < 0 || qy >= pr.H) continue;
            const int qx0 = x + pr.kw / 2;                                   // the query of w = 0; w steps it down
            const long long qrow0 = ((static_cast<long long>(qt) * pr.H + qy) * pr.W + qx0) * pr.heads + m;
            const T* qp = q + qrow0 * D + ch;
            const T* dp = dout + qrow0 * D + ch;
            const float2* cp = coef + qrow0 * pr.P + (u * pr.kh + vv) * pr.kw;
            for (int w = 0; w < pr.kw; ++w, qp -= tok, dp -= tok, cp -= coef_tok - 1) {
                const int qx = qx0 - w;
                if (qx < 0 || qx >= pr.W) continue;
                const float2 c = __ldg(cp);
                const Row qr = E::load(qp);
                const Row dr = E::load(dp);
                E::axpy_paired(c.x, qr, ak);
                E::axpy_paired(c.y, dr, av);
            }
        }
    }
    const long long row = n * pr.heads + m;
    E::store(dk + row * D + ch, ak);
    E::store(dv + row * D + ch, av);
}

template <typename T, int D>
cudaError_t launch_t(const void* q, const void* k, const void* v, const float* lse, const void* dout, void* dq,
                     void* dk, void* dv, float* doffsets, float2* coef, const float* table, const Problem& pr,
                     bool tile_grad, cudaStream_t stream) {
    constexpr int LPR = D / Elt<T, 1>::VEC;
    const int box = (doffsets || table) ? (pr.kt + 1) * (pr.kh + 1) * (pr.kw + 1) : pr.P;
    const size_t box8 = static_cast<size_t>((box + 7) & ~7);
    const size_t per_group = (2 * box8 + 2 * pr.P) * sizeof(float);
    const size_t tables = box8 * sizeof(int4) + static_cast<size_t>((pr.P + 3) & ~3) * sizeof(int);
    int threads = 256;
    while (threads > 32 && tables + static_cast<size_t>(threads / LPR) * (per_group + sizeof(long long)) > 64 * 1024) threads /= 2;
    const size_t smem = tables + static_cast<size_t>(threads / LPR) * (per_group + sizeof(long long));   // + a position per group
    auto qk = fixed_window_backward_query_kernel<T, D, false>;
    if (table) {
        qk = fixed_window_backward_query_kernel<T, D, true>;
        // measured: the compile-time window pays for (2,2,2) only (backward 5.36 -> 4.94 ms on the sweep grid); the
        // instances for (3,3,3), (3,5,5) and (3,7,7) were 3 to 13 % slower than the generic kernel
        if (pr.kt == 2 && pr.kh == 2 && pr.kw == 2) qk = fixed_window_backward_query_kernel<T, D, true, 2, 2, 2>;
    }
    if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(qk, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    long long groups = threads / LPR;
    long long blocks = (pr.items + groups - 1) / groups;
    // bf16: dQ, dK and dV per tile, after the coefficients are out - from regions in shared memory for the
    // small windows, as plane-by-plane products on the tensor cores for the larger ones
    const bool planes = std::is_same<T, __nv_bfloat16>::value && tile_grad && fixed_window_planes_grad_covers(pr, true);
    const bool tiled = planes || (std::is_same<T, __nv_bfloat16>::value && tile_grad && fixed_window_tile_grad_covers(pr, true));
    qk<<<static_cast<unsigned>(blocks), threads, smem, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), lse, static_cast<const T*>(dout),
        tiled ? nullptr : static_cast<T*>(dq), doffsets, coef, table, planes, pr);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (tiled) {
        if (planes ? try_fixed_window_planes_grad(q, k, dout, reinterpret_cast<const float*>(coef), dq, dk, dv, pr, stream, &e)
                   : try_fixed_window_tile_grad(q, k, dout, coef, dq, dk, dv, pr, stream, &e))
            return e;
        // could not be launched after all: the query kernel once more, this time with its dQ (and the
        // coefficients in the order the key kernel reads them)
        qk<<<static_cast<unsigned>(blocks), threads, smem, stream>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), lse, static_cast<const T*>(dout),
            static_cast<T*>(dq), doffsets, coef, table, false, pr);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    groups = 256 / LPR;
    blocks = (pr.items + groups - 1) / groups;
    fixed_window_backward_key_kernel<T, D><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(dout), coef, static_cast<T*>(dk), static_cast<T*>(dv), pr);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fixed_window_backward(const void* q, const void* k, const void* v, const float* lse,
                                         const void* dout, void* dq, void* dk, void* dv, float* doffsets,
                                         float2* coef, const float* table, const Problem& pr, bool bf16,
                                         bool tile_grad, cudaStream_t stream) {
#define DSA3D_CASE(DD)                                                                                                 \
    case DD:                                                                                                           \
        return bf16 ? launch_t<__nv_bfloat16, DD>(q, k, v, lse, dout, dq, dk, dv, doffsets, coef, table, pr, tile_grad, stream)   \
                    : launch_t<float, DD>(q, k, v, lse, dout, dq, dk, dv, doffsets, coef, table, pr, tile_grad, stream);
    switch (pr.d) {
        DSA3D_CASE(32)
        DSA3D_CASE(64)
        DSA3D_CASE(128)
    }
#undef DSA3D_CASE
    return cudaErrorInvalidValue;
}

}  // namespace dsa3d
