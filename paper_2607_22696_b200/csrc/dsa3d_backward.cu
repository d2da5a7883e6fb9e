// Backward of 3D Deformable Slide Attention: dQ, dK, dV and dOffsets.
//
// Same work decomposition as the forward: a group of LPR = d / VEC lanes owns one
// (token, head) item, items are ordered head-major.  The sampling weights are recomputed
// from the offsets, the softmax weights from the saved lse; nothing of size N*P*d exists.
//
// Pass 1 (gather): for every sample the corner rows of K and V are loaded once; the lane
//   partials of  s = sum_c w_c (q.K_c),  g = sum_c w_c (dO.V_c)  and of the six
//   derivative sums  A_a = sum_c (dw_c/da)(q.K_c),  B_a = sum_c (dw_c/da)(dO.V_c)  are
//   reduced over the group; alpha_p = exp(s_p - lse).  With delta = sum_p alpha_p g_p,
//   dQ = scale * (sum_p alpha_p g_p k_p - delta * sum_p alpha_p k_p) needs no second look
//   at K.  The eight per-sample numbers are parked in shared memory.
// Pass 2 (scatter): dS_p = alpha_p (g_p - delta);
//   dOffsets[p, a] = scale dS_p A_a + alpha_p B_a;  for each corner with a non-zero weight
//   dK[corner] += w_c scale dS_p q  and  dV[corner] += w_c alpha_p dO  go to the fp32
//   accumulators with 16-byte vector reductions (red.global.add.v4.f32).
#include "dsa3d_common.cuh"
#include "dsa3d_kernels.h"

namespace dsa3d {

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

constexpr int kStats = 8;   // per sample: alpha, g, A_t, A_y, A_x, B_t, B_y, B_x

template <typename T, int D>
__global__ void __launch_bounds__(256)
backward_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                const float* __restrict__ offsets, const float* __restrict__ lse,
                const T* __restrict__ dout, T* __restrict__ dq, float* __restrict__ acc_dk,
                float* __restrict__ acc_dv, float* __restrict__ doffsets, const Problem pr) {
    constexpr int VEC = Elt<T>::VEC;
    constexpr int LPR = D / VEC;
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31;
    const int gl = lane & (LPR - 1);
    const unsigned gmask = group_mask<LPR>(lane);
    const long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    if (item >= pr.items) return;
    float* stats = smem + static_cast<size_t>(threadIdx.x / LPR) * pr.P * kStats;   // [P][8] of this group

    const int m = static_cast<int>(item / pr.N);
    const long long n = item - static_cast<long long>(m) * pr.N;
    const int x = static_cast<int>(n % pr.W);
    const int y = static_cast<int>((n / pr.W) % pr.H);
    const int t = static_cast<int>(n / (static_cast<long long>(pr.W) * pr.H));
    const int HW = pr.H * pr.W;
    const long long row = n * pr.heads + m;
    const int ch = gl * VEC;
    const float scale = rsqrtf(static_cast<float>(D));

    float qf[VEC], dof[VEC];
    Elt<T>::load(q + row * D + ch, qf);
    Elt<T>::load(dout + row * D + ch, dof);
    const float lse2 = __ldg(lse + row) * kLog2e;            // lse in log2 units
    const float* off_row = offsets + row * pr.P * 3;
    const long long tok_stride = static_cast<long long>(pr.heads) * D;
    const long long head_off = static_cast<long long>(m) * D + ch;
    const T* kh = k + head_off;
    const T* vh = v + head_off;

    float u_acc[VEC], kbar[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) u_acc[e] = kbar[e] = 0.0f;
    float delta = 0.0f;

    // ---------------------------------------------------------------- pass 1: gather
    for (int pb = 0; pb < pr.P; pb += LPR) {
        Sample mine;
        mine.base = 0; mine.mask = 0u; mine.ft = mine.fy = mine.fx = 0.0f;
        if (pb + gl < pr.P) mine = make_sample(pr, t, y, x, pb + gl, off_row + (pb + gl) * 3);
        const int cnt = min(LPR, pr.P - pb);
        for (int j = 0; j < cnt; ++j) {
            const Sample s = group_bcast<LPR>(mine, j, gmask);
            const float wt[2] = {1.0f - s.ft, s.ft}, wy[2] = {1.0f - s.fy, s.fy}, wx[2] = {1.0f - s.fx, s.fx};
            float r[kStats];
#pragma unroll
            for (int i = 0; i < kStats; ++i) r[i] = 0.0f;
            float kp[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) kp[e] = 0.0f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int ct = c >> 2, cy = (c >> 1) & 1, cx = c & 1;
                const float w = wt[ct] * wy[cy] * wx[cx];
                const float dwt = (ct ? 1.0f : -1.0f) * wy[cy] * wx[cx];
                const float dwy = (cy ? 1.0f : -1.0f) * wt[ct] * wx[cx];
                const float dwx = (cx ? 1.0f : -1.0f) * wt[ct] * wy[cy];
                const bool needed = (w != 0.0f) | (dwt != 0.0f) | (dwy != 0.0f) | (dwx != 0.0f);
                if (((s.mask >> c) & 1u) && needed) {
                    const int tok = s.base + ct * HW + cy * pr.W + cx;
                    float kk[VEC], vv[VEC];
                    Elt<T>::load(kh + tok * tok_stride, kk);
                    Elt<T>::load(vh + tok * tok_stride, vv);
                    float a = 0.0f, b = 0.0f;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        a = fmaf(qf[e], kk[e], a);
                        b = fmaf(dof[e], vv[e], b);
                        kp[e] = fmaf(w, kk[e], kp[e]);
                    }
                    r[0] = fmaf(w, a, r[0]);
                    r[1] = fmaf(w, b, r[1]);
                    r[2] = fmaf(dwt, a, r[2]);
                    r[3] = fmaf(dwy, a, r[3]);
                    r[4] = fmaf(dwx, a, r[4]);
                    r[5] = fmaf(dwt, b, r[5]);
                    r[6] = fmaf(dwy, b, r[6]);
                    r[7] = fmaf(dwx, b, r[7]);
                }
            }
#pragma unroll
            for (int i = 0; i < kStats; ++i) r[i] = group_sum<LPR>(r[i], gmask);
            const float alpha = exp2f(fmaf(r[0], scale * kLog2e, -lse2));
            const float g = r[1];
            const float ag = alpha * g;
            delta += ag;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                u_acc[e] = fmaf(ag, kp[e], u_acc[e]);
                kbar[e] = fmaf(alpha, kp[e], kbar[e]);
            }
            if (gl == 0) {
                float* st = stats + (pb + j) * kStats;
                st[0] = alpha; st[1] = g;
                st[2] = r[2]; st[3] = r[3]; st[4] = r[4];
                st[5] = r[5]; st[6] = r[6]; st[7] = r[7];
            }
        }
    }
    {
        float dqv[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) dqv[e] = scale * fmaf(-delta, kbar[e], u_acc[e]);
        Elt<T>::store(dq + row * D + ch, dqv);
    }
    __syncwarp(gmask);

    // ---------------------------------------------------------------- pass 2: scatter
    float* dk_h = acc_dk + head_off;
    float* dv_h = acc_dv + head_off;
    float* doff_row = doffsets + row * pr.P * 3;
    for (int pb = 0; pb < pr.P; pb += LPR) {
        Sample mine;
        mine.base = 0; mine.mask = 0u; mine.ft = mine.fy = mine.fx = 0.0f;
        float my_ck = 0.0f, my_cv = 0.0f;
        if (pb + gl < pr.P) {
            const int p = pb + gl;
            mine = make_sample(pr, t, y, x, p, off_row + p * 3);
            const float* st = stats + p * kStats;
            const float alpha = st[0];
            const float dS = alpha * (st[1] - delta);
            my_ck = scale * dS;
            my_cv = alpha;
            doff_row[p * 3 + 0] = fmaf(my_ck, st[2], alpha * st[5]);
            doff_row[p * 3 + 1] = fmaf(my_ck, st[3], alpha * st[6]);
            doff_row[p * 3 + 2] = fmaf(my_ck, st[4], alpha * st[7]);
        }
        const int cnt = min(LPR, pr.P - pb);
        for (int j = 0; j < cnt; ++j) {
            const Sample s = group_bcast<LPR>(mine, j, gmask);
            const float ck = __shfl_sync(gmask, my_ck, j, LPR);
            const float cv = __shfl_sync(gmask, my_cv, j, LPR);
            if (s.mask == 0u) continue;
            const float wt[2] = {1.0f - s.ft, s.ft}, wy[2] = {1.0f - s.fy, s.fy}, wx[2] = {1.0f - s.fx, s.fx};
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float w = wt[c >> 2] * wy[(c >> 1) & 1] * wx[c & 1];
                if (((s.mask >> c) & 1u) && w != 0.0f) {
                    const int tok = s.base + (c >> 2) * HW + ((c >> 1) & 1) * pr.W + (c & 1);
                    const float wk = w * ck, wv = w * cv;
                    float* pk = dk_h + tok * tok_stride;
                    float* pv = dv_h + tok * tok_stride;
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

template <typename T, int D>
static cudaError_t launch_backward_t(const void* q, const void* k, const void* v, const float* offsets,
                                     const float* lse, const void* dout, void* dq, float* acc_dk,
                                     float* acc_dv, float* doffsets, const Problem& pr,
                                     cudaStream_t stream) {
    constexpr int LPR = D / Elt<T>::VEC;
    // Shared memory holds 8 floats per (group, sample); shrink the block for large windows.
    int threads = 256;
    while (threads > 32 && static_cast<size_t>(threads / LPR) * pr.P * kStats * sizeof(float) > 64 * 1024)
        threads /= 2;
    const size_t smem = static_cast<size_t>(threads / LPR) * pr.P * kStats * sizeof(float);
    auto kern = backward_kernel<T, D>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    const long long groups_per_block = threads / LPR;
    const long long blocks = (pr.items + groups_per_block - 1) / groups_per_block;
    kern<<<static_cast<unsigned>(blocks), threads, smem, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), offsets, lse,
        static_cast<const T*>(dout), static_cast<T*>(dq), acc_dk, acc_dv, doffsets, pr);
    return cudaGetLastError();
}

cudaError_t launch_backward(const void* q, const void* k, const void* v, const float* offsets,
                            const float* lse, const void* dout, void* dq, float* acc_dk, float* acc_dv,
                            float* doffsets, const Problem& pr, bool bf16, cudaStream_t stream) {
#define DSA3D_CASE(DD)                                                                                   \
    case DD:                                                                                             \
        return bf16 ? launch_backward_t<__nv_bfloat16, DD>(q, k, v, offsets, lse, dout, dq, acc_dk,     \
                                                           acc_dv, doffsets, pr, stream)                 \
                    : launch_backward_t<float, DD>(q, k, v, offsets, lse, dout, dq, acc_dk, acc_dv,      \
                                                   doffsets, pr, stream);
    switch (pr.d) {
        DSA3D_CASE(32)
        DSA3D_CASE(64)
        DSA3D_CASE(128)
    }
#undef DSA3D_CASE
    return cudaErrorInvalidValue;
}

__global__ void __launch_bounds__(256)
convert_bf16_kernel(const float4* __restrict__ acc, uint2* __restrict__ dst, long long count4) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < count4; i += stride) {
        const float4 a = acc[i];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(a.z, a.w);
        dst[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
}

cudaError_t launch_convert_bf16(const float* acc, void* dst, long long count, cudaStream_t stream) {
    const long long count4 = count / 4;      // d is a multiple of 32, so count is a multiple of 4
    long long blocks = (count4 + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    if (blocks < 1) blocks = 1;
    convert_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(acc), reinterpret_cast<uint2*>(dst), count4);
    return cudaGetLastError();
}

}  // namespace dsa3d
