// Shared device helpers of the 3D-DSA kernels: problem description, element access for
// fp32 / bf16 storage, sample geometry (Formulation: position = token coordinate + window
// displacement + learned offset; trilinear corners with zero padding) and group shuffles.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dsa3d {

struct Problem {
    int T, H, W, heads, d;
    int kt, kh, kw, P;
    long long N;       // T*H*W
    long long items;   // N*heads: one work item per (token, head)
};

// ---------------------------------------------------------------------------------------
// Element access.  A "vector" is 16 bytes: 8 bf16 or 4 fp32 channels.
// ---------------------------------------------------------------------------------------
template <typename T> struct Elt;

template <> struct Elt<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void load(const float* p, float (&x)[4]) {
        const float4 r = __ldg(reinterpret_cast<const float4*>(p));
        x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&x)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};

template <> struct Elt<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[8]) {
        const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {           // bf16 is the upper half of an fp32
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);   // RNE
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// ---------------------------------------------------------------------------------------
// Sample geometry.  `base` is the token index of corner (0,0,0) (it may be "virtual",
// i.e. have a component of -1; only corners flagged in `mask` are ever dereferenced),
// bit c = ct*4 + cy*2 + cx of `mask` says corner c lies inside the grid, f* are the
// fractional parts.  A sample with a NaN position or one at < -1 or >= size on any axis
// has mask 0.  The position is float(coord + b) + offset with one fp32 rounding, then
// floorf, then the fp32 difference: the same sequence on every path so that the integer
// cell decision never depends on who computes it.
// ---------------------------------------------------------------------------------------
struct Sample {
    int base;
    unsigned mask;
    float ft, fy, fx;
};

__device__ __forceinline__ bool axis_cell(int coord_plus_b, float off, int size, int& i0, float& f,
                                          unsigned& lo_ok, unsigned& hi_ok) {
    const float pi = __fadd_rn(static_cast<float>(coord_plus_b), off);
    if (!(pi >= -1.0f) || !(pi < static_cast<float>(size))) return false;
    const float fl = floorf(pi);
    i0 = static_cast<int>(fl);
    f = __fsub_rn(pi, fl);
    lo_ok = i0 >= 0;
    hi_ok = i0 + 1 <= size - 1;
    return true;
}

__device__ __forceinline__ Sample make_sample(const Problem& pr, int t, int y, int x, int p,
                                              const float* __restrict__ off3) {
    const int w = p % pr.kw;
    const int v = (p / pr.kw) % pr.kh;
    const int u = p / (pr.kw * pr.kh);
    Sample s;
    s.base = 0; s.mask = 0u; s.ft = s.fy = s.fx = 0.0f;
    int it, iy, ix;
    unsigned t0, t1, y0, y1, x0, x1;
    float ft, fy, fx;
    const float ot = __ldg(off3), oy = __ldg(off3 + 1), ox = __ldg(off3 + 2);
    if (!axis_cell(t + u - pr.kt / 2, ot, pr.T, it, ft, t0, t1)) return s;
    if (!axis_cell(y + v - pr.kh / 2, oy, pr.H, iy, fy, y0, y1)) return s;
    if (!axis_cell(x + w - pr.kw / 2, ox, pr.W, ix, fx, x0, x1)) return s;
    s.base = (it * pr.H + iy) * pr.W + ix;
    s.ft = ft; s.fy = fy; s.fx = fx;
    unsigned m = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const unsigned ok = ((c & 4) ? t1 : t0) & ((c & 2) ? y1 : y0) & ((c & 1) ? x1 : x0);
        m |= ok << c;
    }
    s.mask = m;
    return s;
}

// Shuffles inside a group of LPR consecutive lanes (LPR a power of two <= 32).
template <int LPR> __device__ __forceinline__ unsigned group_mask(int lane) {
    if constexpr (LPR == 32) {
        return 0xffffffffu;
    } else {
        return ((1u << LPR) - 1u) << (lane & ~(LPR - 1));
    }
}

template <int LPR> __device__ __forceinline__ float group_sum(float v, unsigned gmask) {
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(gmask, v, o, LPR);
    return v;
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

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace dsa3d
