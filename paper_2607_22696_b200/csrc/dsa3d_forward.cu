// Forward of 3D Deformable Slide Attention (Eq. 1 second term and the softmax under it).
//
// One group of LPR = d / VEC lanes owns one (token, head) item; each lane holds VEC
// consecutive channels (16 bytes) of every row it touches.  Work items are ordered
// head-major (item = head * N + token) so that the CTAs in flight at any time gather from
// one head's K/V over a few neighbouring frames, which is what keeps the corner gathers in
// L2.  Per sample: the 8 corner rows of K and of V are loaded with 16-byte loads, the
// logit is the weighted sum of the corner dot products, and the output is accumulated with
// an online softmax in fp32 registers; nothing of size N*P is written.
//
// A sample whose 8 corners are all inside the grid with non-zero weights (the usual case
// for real-valued offsets) takes a branch-free path that issues its 16 row loads back to
// back; border samples and samples on integer positions take a per-corner path that skips
// corners outside the grid and corners of weight zero.
#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"

namespace dsa3d {

__device__ const float kZeroOffset[3] = {0.0f, 0.0f, 0.0f};     // stands in for a NULL offsets tensor

#ifndef DSA3D_FWD_MINBLOCKS
#define DSA3D_FWD_MINBLOCKS 3
#endif

template <typename T, int D, int NV, bool kAdd>
__global__ void __launch_bounds__(256, NV == 2 ? 2 : DSA3D_FWD_MINBLOCKS)
forward_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
               const float* __restrict__ offsets, const T* addend, T* out, float* __restrict__ lse,
               const Problem pr, const int* __restrict__ gate) {
    if (gate && *gate == 0) return;                      // another kernel takes this call (see launch_forward)
    using E = Elt<T, NV>;
    using Row = typename E::Row;
    constexpr int VEC = E::VEC;
    constexpr int LPR = D / VEC;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (LPR - 1);
    constexpr unsigned gmask = kFullMask;
    long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    const long long warp_first = (static_cast<long long>(blockIdx.x) * blockDim.x + (threadIdx.x & ~31)) / LPR;
    if (warp_first >= pr.items) return;                  // whole warp past the end
    const bool active = item < pr.items;                 // a trailing group repeats the last item, stores off
    if (!active) item = pr.items - 1;

    const int m = static_cast<int>(item / pr.q_count);
    const long long n = pr.q_begin + (item - static_cast<long long>(m) * pr.q_count);
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const long long row = (n * pr.heads + m);               // row index into [N*heads, ...]
    const int ch = gl * VEC;
    const long long tok_stride = static_cast<long long>(pr.heads) * D;
    const long long sx = tok_stride;                         // element stride between x neighbours
    const long long sy = static_cast<long long>(pr.W) * sx;      // 64-bit once, so that the pointer
    const long long st = static_cast<long long>(pr.H) * sy;      // arithmetic below needs no widening                                // < 2^31: checked by the host

    const Row qr = E::load(q + row * D + ch);
    const float lscale = rsqrtf(static_cast<float>(D)) * kLog2e;    // logits in log2 units
    const float* off_row = offsets + row * pr.P * 3;
    const T* kh = k + static_cast<long long>(m) * D + ch;    // + tok * heads * D
    const long long v_minus_k = v - k;                       // same layout: V row = K row + this
    [[maybe_unused]] const long long kv_extent = pr.N * pr.heads * D;      // elements of K (= of V): checked build

    float acc[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[j] = 0.0f;
    float m_run = -INFINITY, l_run = 0.0f;

    for (int pb = 0; pb < pr.P; pb += LPR) {
        Sample mine;
        mine.base = 0; mine.mask = 0u; mine.ft = mine.fy = mine.fx = 0.0f;
        if (pb + gl < pr.P)
            mine = to_sample(pr, make_cell(pr, t, y, x, pb + gl, offsets ? off_row + (pb + gl) * 3 : kZeroOffset));
        const int cnt = min(LPR, pr.P - pb);
        if constexpr (LPR >= 8) {
            // Fixed-window regime: every sample of this chunk (in every group of the warp) sits
            // exactly on a grid position, so it needs one K row and one V row.  Eight samples
            // are then taken together - 16 loads in flight instead of 2 - and their eight
            // logits leave one transposed reduction.
            const bool lattice = pb + gl >= pr.P || (mine.ft == 0.0f && mine.fy == 0.0f && mine.fx == 0.0f);
            if (__all_sync(kFullMask, lattice)) {
                for (int jb = 0; jb < cnt; jb += 8) {
                    Row kk[8], vv[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int base = __shfl_sync(gmask, mine.base, jb + i, LPR);
                        const unsigned mk = __shfl_sync(gmask, mine.mask, jb + i, LPR);
                        kk[i] = E::zero();
                        vv[i] = E::zero();
                        if ((mk & 1u) && jb + i < cnt) {            // corner (0,0,0) inside the grid
                            const T* pk = kh + base * tok_stride;
                            if (DSA3D_IN_RANGE(pr, pk - k, kv_extent, 1)) {
                                kk[i] = E::load(pk);
                                vv[i] = E::load(pk + v_minus_k);
                            }
                        }
                    }
                    float dd[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) dd[i] = E::dot(qr, kk[i], 0.0f);
                    group_reduce8<LPR>(dd, gl, gmask);
                    float sp[8], mx = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        sp[i] = __shfl_sync(gmask, dd[0], reduce8_lane<LPR>(i), LPR) * lscale;
                        if (jb + i >= cnt) sp[i] = -INFINITY;       // no such sample
                        mx = fmaxf(mx, sp[i]);
                    }
                    if (mx > m_run + 8.0f) {
                        const float corr = exp2f(m_run - mx);
                        l_run *= corr;
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[e] *= corr;
                        m_run = mx;
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float pe = exp2f(sp[i] - m_run);
                        l_run += pe;
                        E::axpy(pe, vv[i], acc);
                    }
                }
                continue;
            }
        }
        for (int j = 0; j < cnt; ++j) {
            const Sample s = group_bcast<LPR>(mine, j, gmask);
            const float wt[2] = {1.0f - s.ft, s.ft}, wy[2] = {1.0f - s.fy, s.fy}, wx[2] = {1.0f - s.fx, s.fx};
            float w[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) w[c] = wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1];
            // corner row pointers: (ct, cy) pairs, the cx = 1 row is one token further
            const T* kp4[4];
            kp4[0] = kh + s.base * tok_stride;
            kp4[1] = kp4[0] + sy;
            kp4[2] = kp4[0] + st;
            kp4[3] = kp4[2] + sy;
            const bool full = s.mask == 0xffu && s.ft != 0.0f && s.fy != 0.0f && s.fx != 0.0f;
            float sdot = 0.0f;
            Row vv[8];
            if (full) {
                Row kk[8];
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    kk[c] = DSA3D_IN_RANGE(pr, kp4[c >> 1] + (c & 1) * sx - k, kv_extent, 2) ? E::load(kp4[c >> 1] + (c & 1) * sx) : E::zero();
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    vv[c] = DSA3D_IN_RANGE(pr, kp4[c >> 1] + (c & 1) * sx - k, kv_extent, 2) ? E::load(kp4[c >> 1] + (c & 1) * sx + v_minus_k) : E::zero();
#pragma unroll
                for (int c = 0; c < 8; ++c) sdot = fmaf(w[c], E::dot(qr, kk[c], 0.0f), sdot);
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    vv[c] = E::zero();
                    if (((s.mask >> c) & 1u) && w[c] != 0.0f && DSA3D_IN_RANGE(pr, kp4[c >> 1] + (c & 1) * sx - k, kv_extent, 3)) {
                        const T* pk = kp4[c >> 1] + (c & 1) * sx;
                        const Row kk = E::load(pk);
                        vv[c] = E::load(pk + v_minus_k);
                        sdot = fmaf(w[c], E::dot(qr, kk, 0.0f), sdot);
                    } else {
                        w[c] = 0.0f;
                    }
                }
            }
            const float sp = group_sum<LPR>(sdot, gmask) * lscale;
            // Online softmax with a lazily updated reference: the running maximum m_run only
            // moves when a logit exceeds it by more than 8 (log2 units), so exp2(sp - m_run)
            // stays below 256 and the accumulators are rescaled only a few times per query.
            if (sp > m_run + 8.0f) {
                const float corr = exp2f(m_run - sp);
                l_run *= corr;
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] *= corr;
                m_run = sp;
            }
            const float pe = exp2f(sp - m_run);
            l_run += pe;
#pragma unroll
            for (int c = 0; c < 8; ++c) E::axpy(pe * w[c], vv[c], acc);
        }
    }
    const float inv = 1.0f / l_run;
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] *= inv;
    if (active) {
        if constexpr (kAdd) {                            // first term of Eq. 1, added before the rounding
            float add[VEC];
            E::to_float(E::load(addend + row * D + ch), add);
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] += add[e];
        }
        E::store(out + row * D + ch, acc);
        if (gl == 0) lse[row] = (m_run + log2f(l_run)) * kLn2;
    }
}

// 16-byte vectors per lane.  One everywhere: two (8 lanes per 128-channel bf16 item) halves
// the per-item bookkeeping but costs a block of occupancy, which the forward loses more by.
#ifndef DSA3D_FWD_BF16_NV
#define DSA3D_FWD_BF16_NV 1
#endif
template <typename T, int D> struct FwdLaneWidth { static constexpr int NV = 1; };
template <> struct FwdLaneWidth<__nv_bfloat16, 128> { static constexpr int NV = DSA3D_FWD_BF16_NV; };

template <typename T, int D>
static cudaError_t launch_forward_t(const void* q, const void* k, const void* v, const float* offsets,
                                    const void* addend, void* out, float* lse, const Problem& pr,
                                    cudaStream_t stream, const int* gate) {
    constexpr int NV = FwdLaneWidth<T, D>::NV;
    constexpr int LPR = D / Elt<T, NV>::VEC;
    constexpr int threads = 256;
    const long long groups_per_block = threads / LPR;
    const long long blocks = (pr.items + groups_per_block - 1) / groups_per_block;
    if (addend)
        forward_kernel<T, D, NV, true><<<static_cast<unsigned>(blocks), threads, 0, stream>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), offsets,
            static_cast<const T*>(addend), static_cast<T*>(out), lse, pr, gate);
    else
        forward_kernel<T, D, NV, false><<<static_cast<unsigned>(blocks), threads, 0, stream>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), offsets, nullptr,
            static_cast<T*>(out), lse, pr, gate);
    return cudaGetLastError();
}

cudaError_t launch_forward(const void* q, const void* k, const void* v, const float* offsets, const void* addend,
                           void* out, float* lse, const Problem& pr, bool bf16, cudaStream_t stream, const int* gate) {
#define DSA3D_CASE(DD)                                                                                    \
    case DD:                                                                                              \
        return bf16 ? launch_forward_t<__nv_bfloat16, DD>(q, k, v, offsets, addend, out, lse, pr, stream, gate)   \
                    : launch_forward_t<float, DD>(q, k, v, offsets, addend, out, lse, pr, stream, gate);
    switch (pr.d) {
        DSA3D_CASE(32)
        DSA3D_CASE(64)
        DSA3D_CASE(128)
    }
#undef DSA3D_CASE
    return cudaErrorInvalidValue;
}

}  // namespace dsa3d
