// C ABI of the 3D-DSA library: argument validation, workspace layout, launches.
// Declarations and the contract of every entry point are in include/dsa3d.h.
#include <stdint.h>

#include "../../include/dsa3d.h"
#include "dsa3d_kernels.h"

namespace {

thread_local int g_last_cuda_error = 0;
thread_local cudaEvent_t g_events[4] = {nullptr, nullptr, nullptr, nullptr};   // fwd start/stop, bwd start/stop

cudaError_t record(int which, cudaStream_t stream) {
    return g_events[which] ? cudaEventRecord(g_events[which], stream) : cudaSuccess;
}

int cuda_failed(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return DSA3D_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Fills `pr`; returns DSA3D_OK or the reason the shape is rejected.
int make_problem(int T, int H, int W, int heads, int d, const int* window, int dtype, dsa3d::Problem& pr) {
    if (!window) return DSA3D_ERR_NULL_POINTER;
    if (T < 1 || H < 1 || W < 1 || heads < 1 || d < 1) return DSA3D_ERR_BAD_SHAPE;
    if (window[0] < 1 || window[1] < 1 || window[2] < 1) return DSA3D_ERR_BAD_SHAPE;
    const long long N = static_cast<long long>(T) * H * W;
    if (N >= (1LL << 31)) return DSA3D_ERR_BAD_SHAPE;
    if (dtype != DSA3D_F32 && dtype != DSA3D_BF16) return DSA3D_ERR_UNSUPPORTED;
    if (d != 32 && d != 64 && d != 128) return DSA3D_ERR_UNSUPPORTED;
    const long long P = static_cast<long long>(window[0]) * window[1] * window[2];
    if (P > 256) return DSA3D_ERR_UNSUPPORTED;
    // one CUDA block covers at least 8 items, and the grid has at most 2^31 - 1 blocks
    if (N * heads / 8 >= (1LL << 31) - 1) return DSA3D_ERR_BAD_SHAPE;
    pr.T = T; pr.H = H; pr.W = W; pr.heads = heads; pr.d = d;
    pr.kt = window[0]; pr.kh = window[1]; pr.kw = window[2];
    pr.P = static_cast<int>(P);
    pr.N = N;
    pr.items = N * heads;
    return DSA3D_OK;
}

}  // namespace

extern "C" {

int dsa3d_forward(const void* q, const void* k, const void* v, const float* offsets, int T, int H, int W,
                  int heads, int d, const int window[3], void* out, float* lse, int dtype, void* stream) {
    if (!q || !k || !v || !offsets || !out || !lse) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(out) ||
        !aligned16(lse))
        return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = record(0, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = dsa3d::launch_forward(q, k, v, offsets, out, lse, pr, dtype == DSA3D_BF16, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(1, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

size_t dsa3d_backward_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    if (dtype == DSA3D_F32) return 0;
    return static_cast<size_t>(pr.items) * pr.d * sizeof(float) * 2;   // fp32 dK and dV accumulators
}

int dsa3d_backward(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                   const void* dout, int T, int H, int W, int heads, int d, const int window[3], void* dq,
                   void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes, int dtype,
                   void* stream_) {
    if (!q || !k || !v || !offsets || !lse || !dout || !dq || !dk || !dv || !doffsets)
        return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(lse) ||
        !aligned16(dout) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(doffsets))
        return DSA3D_ERR_MISALIGNED;
    const size_t need = dsa3d_backward_workspace_bytes(T, H, W, heads, d, window, dtype);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return DSA3D_ERR_WORKSPACE;
        if (!aligned16(workspace)) return DSA3D_ERR_MISALIGNED;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const bool bf16 = dtype == DSA3D_BF16;
    const size_t count = static_cast<size_t>(pr.items) * pr.d;
    float* acc_dk = bf16 ? static_cast<float*>(workspace) : static_cast<float*>(dk);
    float* acc_dv = bf16 ? static_cast<float*>(workspace) + count : static_cast<float*>(dv);
    cudaError_t e;
    if (bf16) {
        e = cudaMemsetAsync(workspace, 0, need, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    } else {
        e = cudaMemsetAsync(dk, 0, count * sizeof(float), stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaMemsetAsync(dv, 0, count * sizeof(float), stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    e = record(2, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    e = dsa3d::launch_backward(q, k, v, offsets, lse, dout, dq, acc_dk, acc_dv, doffsets, pr, bf16, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(3, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    if (bf16) {
        e = dsa3d::launch_convert_bf16(acc_dk, dk, static_cast<long long>(count), stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = dsa3d::launch_convert_bf16(acc_dv, dv, static_cast<long long>(count), stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return DSA3D_OK;
}

namespace {

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Layout of the device arena of dsa3d_step_host: offsets of each buffer, total in `total`.
struct Arena {
    size_t q, k, v, dout, out, dq, dk, dv, offsets, doffsets, lse, workspace, total;
    size_t row_bytes, off_bytes, lse_bytes, ws_bytes;
};

Arena arena_layout(const dsa3d::Problem& pr, int dtype) {
    Arena a;
    const size_t elt = dtype == DSA3D_BF16 ? 2 : 4;
    a.row_bytes = static_cast<size_t>(pr.items) * pr.d * elt;
    a.off_bytes = static_cast<size_t>(pr.items) * pr.P * 3 * sizeof(float);
    a.lse_bytes = static_cast<size_t>(pr.items) * sizeof(float);
    a.ws_bytes = dtype == DSA3D_BF16 ? static_cast<size_t>(pr.items) * pr.d * sizeof(float) * 2 : 0;
    size_t at = 0;
    size_t* rows[8] = {&a.q, &a.k, &a.v, &a.dout, &a.out, &a.dq, &a.dk, &a.dv};
    for (size_t* r : rows) { *r = at; at += round256(a.row_bytes); }
    a.offsets = at; at += round256(a.off_bytes);
    a.doffsets = at; at += round256(a.off_bytes);
    a.lse = at; at += round256(a.lse_bytes);
    a.workspace = at; at += round256(a.ws_bytes);
    a.total = at;
    return a;
}

}  // namespace

size_t dsa3d_step_host_arena_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    return arena_layout(pr, dtype).total;
}

int dsa3d_step_host(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                    const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                    void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                    void* arena, size_t arena_bytes, int dtype, void* stream_) {
    if (!q_h || !k_h || !v_h || !offsets_h || !dout_h || !out_h || !lse_h || !dq_h || !dk_h || !dv_h ||
        !doffsets_h || !arena)
        return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return DSA3D_ERR_MISALIGNED;
    const Arena a = arena_layout(pr, dtype);
    if (arena_bytes < a.total) return DSA3D_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char* base = static_cast<char*>(arena);
    const struct { size_t at; const void* src; size_t bytes; } in[5] = {
        {a.q, q_h, a.row_bytes}, {a.k, k_h, a.row_bytes}, {a.v, v_h, a.row_bytes},
        {a.offsets, offsets_h, a.off_bytes}, {a.dout, dout_h, a.row_bytes}};
    for (const auto& c : in) {
        const cudaError_t e = cudaMemcpyAsync(base + c.at, c.src, c.bytes, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    int st = dsa3d_forward(base + a.q, base + a.k, base + a.v, reinterpret_cast<const float*>(base + a.offsets),
                           T, H, W, heads, d, window, base + a.out, reinterpret_cast<float*>(base + a.lse),
                           dtype, stream_);
    if (st != DSA3D_OK) return st;
    st = dsa3d_backward(base + a.q, base + a.k, base + a.v, reinterpret_cast<const float*>(base + a.offsets),
                        reinterpret_cast<const float*>(base + a.lse), base + a.dout, T, H, W, heads, d, window,
                        base + a.dq, base + a.dk, base + a.dv, reinterpret_cast<float*>(base + a.doffsets),
                        a.ws_bytes ? base + a.workspace : nullptr, a.ws_bytes, dtype, stream_);
    if (st != DSA3D_OK) return st;
    const struct { size_t at; void* dst; size_t bytes; } outc[6] = {
        {a.out, out_h, a.row_bytes}, {a.lse, lse_h, a.lse_bytes}, {a.dq, dq_h, a.row_bytes},
        {a.dk, dk_h, a.row_bytes}, {a.dv, dv_h, a.row_bytes}, {a.doffsets, doffsets_h, a.off_bytes}};
    for (const auto& c : outc) {
        const cudaError_t e = cudaMemcpyAsync(c.dst, base + c.at, c.bytes, cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return DSA3D_OK;
}

int dsa3d_set_profile_events(void* fwd_start, void* fwd_stop, void* bwd_start, void* bwd_stop) {
    g_events[0] = static_cast<cudaEvent_t>(fwd_start);
    g_events[1] = static_cast<cudaEvent_t>(fwd_stop);
    g_events[2] = static_cast<cudaEvent_t>(bwd_start);
    g_events[3] = static_cast<cudaEvent_t>(bwd_stop);
    return DSA3D_OK;
}

const char* dsa3d_status_string(int status) {
    switch (status) {
        case DSA3D_OK: return "success";
        case DSA3D_ERR_NULL_POINTER: return "a required pointer is NULL";
        case DSA3D_ERR_BAD_SHAPE: return "invalid grid, head count or window size";
        case DSA3D_ERR_UNSUPPORTED: return "unsupported dtype, head dimension or window";
        case DSA3D_ERR_MISALIGNED: return "a pointer is not 16-byte aligned";
        case DSA3D_ERR_WORKSPACE: return "workspace missing or too small";
        case DSA3D_ERR_CUDA: return "a CUDA runtime call failed";
        default: return "unknown status";
    }
}

int dsa3d_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
