// C ABI of the 3D-DSA library: argument validation, workspace layout, launches.
// Declarations and the contract of every entry point are in include/dsa3d.h.
#include <atomic>
#include <cstdlib>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "../../include/dsa3d.h"
#include "dsa3d_kernels.h"

namespace {

thread_local int g_last_cuda_error = 0;
thread_local cudaEvent_t g_events[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};   // fwd, bwd gather, bwd tile scatter: start/stop each

cudaError_t record(int which, cudaStream_t stream) {
    return g_events[which] ? cudaEventRecord(g_events[which], stream) : cudaSuccess;
}

int cuda_failed(cudaError_t e) { return dsa3d::note_cuda_error(e); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checked build: the word the kernels record their first out-of-range index in.
#ifdef DSA3D_DEBUG
__device__ unsigned long long g_debug_word = 0ull;
unsigned long long* debug_word_address() {
    void* p = nullptr;
    return cudaGetSymbolAddress(&p, g_debug_word) == cudaSuccess ? static_cast<unsigned long long*>(p) : nullptr;
}
#else
unsigned long long* debug_word_address() { return nullptr; }
#endif

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
    pr.inv_kw = ((1u << 20) + static_cast<unsigned>(pr.kw) - 1u) / static_cast<unsigned>(pr.kw);
    pr.inv_kh = ((1u << 20) + static_cast<unsigned>(pr.kh) - 1u) / static_cast<unsigned>(pr.kh);
    // one frame of rows must be addressable with 32-bit element offsets
    if (static_cast<long long>(H) * W * heads * d >= (1LL << 31)) return DSA3D_ERR_BAD_SHAPE;
    pr.P = static_cast<int>(P);
    pr.N = N;
    pr.items = N * heads;
    pr.q_begin = 0;
    pr.q_count = N;
    pr.tile_t = pr.tile_y = pr.tile_x = 0;
    pr.halo = 0;
    pr.tiles_t = pr.tiles_y = pr.tiles_x = 0;
    pr.tt_begin = pr.tt_count = 0;
    pr.key_blocks = 0;
    pr.blk_count = nullptr;
    pr.blk_list = nullptr;
    pr.blk_cap = 0;
    pr.gate = nullptr;
    pr.debug_word = debug_word_address();
    return DSA3D_OK;
}

// Query tiling of the backward scatter: 4 x 8 x 8 queries per tile, halo of 6 cells.  The
// environment variable DSA3D_TILE="tt,ty,tx,halo" overrides it for experiments ("0"
// turns the tile kernel off); values that do not fit shared memory fall back to the default.
constexpr int kTileSlots = 304;          // upper bound on resident tile CTAs (scratch regions)
constexpr size_t kTileSmemLimit = 200 * 1024;

void set_tiling(dsa3d::Problem& pr) {
    int tt = 4, ty = 8, tx = 8, halo = 6;
    if (const char* env = getenv("DSA3D_TILE")) {
        int a = 0, b = 0, c = 0, h = 0;
        const int got = sscanf(env, "%d,%d,%d,%d", &a, &b, &c, &h);
        if (got == 1 && a == 0) return;                       // tiling off
        if (got == 4 && a >= 1 && b >= 1 && c >= 1 && h >= 0 && a * b * c <= 1024) {
            dsa3d::Problem probe = pr;
            probe.tile_t = a; probe.tile_y = b; probe.tile_x = c; probe.halo = h;
            if (dsa3d::tile_smem_bytes(probe) <= kTileSmemLimit) { tt = a; ty = b; tx = c; halo = h; }
        }
    }
    pr.tile_t = tt; pr.tile_y = ty; pr.tile_x = tx; pr.halo = halo;
    pr.tiles_t = (pr.T + tt - 1) / tt;
    pr.tiles_y = (pr.H + ty - 1) / ty;
    pr.tiles_x = (pr.W + tx - 1) / tx;
    pr.tt_begin = 0;
    pr.tt_count = pr.tiles_t;
    // DSA3D_KEY_BLOCKS=1 replaces the tile kernel by the tensor-core key-block kernel where that covers the
    // shape (and no tiling was asked for explicitly): correct and tested, but slower so far.
    const char* kb = getenv("DSA3D_KEY_BLOCKS");
    pr.key_blocks = (kb && kb[0] == '1' && !getenv("DSA3D_TILE") && dsa3d::key_blocks_shape_covered(pr)) ? 1 : 0;
}

struct BackwardWorkspace {
    size_t acc_bytes, coef_bytes, scratch_bytes, total;
    long long entries_per_cta;
};

BackwardWorkspace backward_workspace(const dsa3d::Problem& pr, int dtype, bool tiled) {
    BackwardWorkspace w{};
    if (dtype != DSA3D_BF16) return w;
    w.acc_bytes = static_cast<size_t>(pr.items) * pr.d * sizeof(float) * 2;
    if (tiled && pr.tile_t >= 1) {
        // rounded up so that the 16-byte bin entries behind it stay 16-byte aligned
        w.coef_bytes = (static_cast<size_t>(pr.items) * pr.P * sizeof(float2) + 255) & ~static_cast<size_t>(255);
        if (pr.key_blocks) {
            // per-block counters and sample lists, sorted records of the resident CTAs, in place of the bin entries
            const dsa3d::KeyBlockLayout kb = dsa3d::key_block_layout(pr);
            w.scratch_bytes = kb.count_bytes + kb.list_bytes + kb.sorted_bytes;
        } else {
            w.entries_per_cta = static_cast<long long>(pr.tile_t) * pr.tile_y * pr.tile_x * pr.P * 8;
            w.scratch_bytes = static_cast<size_t>(kTileSlots) * w.entries_per_cta * sizeof(dsa3d::TileEntry);
        }
    }
    w.total = w.acc_bytes + w.coef_bytes + w.scratch_bytes;
    return w;
}

}  // namespace

int dsa3d::note_cuda_error(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return DSA3D_ERR_CUDA;
}

extern "C" {

namespace {
int forward_entry(const void* q, const void* k, const void* v, const float* offsets, const void* addend, int T, int H,
                  int W, int heads, int d, const int window[3], void* out, float* lse, int dtype, void* stream) {
    if (!q || !k || !v || !offsets || !out || !lse) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(out) ||
        !aligned16(lse) || (addend && !aligned16(addend)))
        return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = record(0, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = dsa3d::launch_forward(q, k, v, offsets, addend, out, lse, pr, dtype == DSA3D_BF16, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(1, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}
}  // namespace

int dsa3d_forward(const void* q, const void* k, const void* v, const float* offsets, int T, int H, int W,
                  int heads, int d, const int window[3], void* out, float* lse, int dtype, void* stream) {
    return forward_entry(q, k, v, offsets, nullptr, T, H, W, heads, d, window, out, lse, dtype, stream);
}

int dsa3d_forward_fixed_window(const void* q, const void* k, const void* v, int T, int H, int W, int heads, int d,
                               const int window[3], void* out, float* lse, int dtype, void* stream) {
    if (!q || !k || !v || !out || !lse) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(lse)) return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = record(0, st);
    if (e != cudaSuccess) return cuda_failed(e);
    bool done = false;
    if (dtype == DSA3D_BF16 && !std::getenv("DSA3D_NO_TENSOR_FIXED_WINDOW")) {
        done = dsa3d::try_fixed_window_forward(q, k, v, out, lse, pr, st, &e);
        if (!done) done = dsa3d::try_fixed_window_forward_planes(q, k, v, out, lse, pr, st, &e);
        if (done && e != cudaSuccess) return cuda_failed(e);
    }
    if (!done) {                      // general kernel, a NULL offsets tensor reads as all zeros
        e = dsa3d::launch_forward(q, k, v, nullptr, nullptr, out, lse, pr, dtype == DSA3D_BF16, st);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    e = record(1, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

namespace {
// Gate words of dsa3d_forward_bounded_offsets: one per call, taken round-robin, so that calls whose GPU
// work overlaps (other streams, other threads) do not share one.
constexpr unsigned kGateWords = 1024;
__device__ int g_gate_words[kGateWords];
std::atomic<unsigned> g_next_gate{0};
}  // namespace

int dsa3d_forward_bounded_offsets(const void* q, const void* k, const void* v, const float* offsets, int T, int H, int W,
                                  int heads, int d, const int window[3], void* out, float* lse, int dtype, void* stream) {
    if (!q || !k || !v || !offsets || !out || !lse) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(out) || !aligned16(lse))
        return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = record(0, st);
    if (e != cudaSuccess) return cuda_failed(e);
    bool tiled = false;
    if (dsa3d::bounded_offsets_shape_covered(pr, dtype == DSA3D_BF16) && !std::getenv("DSA3D_NO_TENSOR_FIXED_WINDOW")) {
        void* words = nullptr;
        e = cudaGetSymbolAddress(&words, g_gate_words);
        if (e != cudaSuccess) return cuda_failed(e);
        int* gate = static_cast<int*>(words) + g_next_gate.fetch_add(1u) % kGateWords;
        e = dsa3d::launch_offsets_bound_check(offsets, pr.items * pr.P * 3, gate, st);
        if (e != cudaSuccess) return cuda_failed(e);
        // the tile kernel runs if the check left 0 in the gate, the general kernel if it left 1
        tiled = dsa3d::try_bounded_offsets_forward(q, k, v, offsets, gate, out, lse, pr, st, &e);
        if (tiled && e != cudaSuccess) return cuda_failed(e);
        if (tiled) {
            e = dsa3d::launch_forward(q, k, v, offsets, nullptr, out, lse, pr, true, st, gate);
            if (e != cudaSuccess) return cuda_failed(e);
        }
    }
    if (!tiled) {
        e = dsa3d::launch_forward(q, k, v, offsets, nullptr, out, lse, pr, dtype == DSA3D_BF16, st);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    e = record(1, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

namespace {
bool bounded_backward_tiled(const dsa3d::Problem& pr, int dtype) {
    const char* kb = std::getenv("DSA3D_KEY_BLOCKS");
    return dtype == DSA3D_BF16 && dsa3d::bounded_offsets_backward_covers(pr, true) &&
           !std::getenv("DSA3D_NO_TENSOR_FIXED_WINDOW") && !(kb && kb[0] == '1');
}
}  // namespace

size_t dsa3d_backward_bounded_offsets_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    const size_t general = dsa3d_backward_workspace_bytes(T, H, W, heads, d, window, dtype);
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    if (!bounded_backward_tiled(pr, dtype)) return general;
    const size_t tiled = dsa3d::bounded_offsets_backward_bytes(pr);      // the two routes never hold data at the same time
    return tiled > general ? tiled : general;
}

int dsa3d_backward_bounded_offsets(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                                   const void* dout, int T, int H, int W, int heads, int d, const int window[3], void* dq,
                                   void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes, int dtype,
                                   void* stream) {
    if (!q || !k || !v || !offsets || !lse || !dout || !dq || !dk || !dv || !doffsets) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!bounded_backward_tiled(pr, dtype))
        return dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets, workspace,
                                    workspace_bytes, dtype, stream, true);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(lse) || !aligned16(dout) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(doffsets))
        return DSA3D_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < dsa3d_backward_bounded_offsets_workspace_bytes(T, H, W, heads, d, window, dtype))
        return DSA3D_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* words = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&words, g_gate_words);
    if (e != cudaSuccess) return cuda_failed(e);
    int* gate = static_cast<int*>(words) + g_next_gate.fetch_add(1u) % kGateWords;
    e = dsa3d::launch_offsets_bound_check(offsets, pr.items * pr.P * 3, gate, st);
    if (e != cudaSuccess) return cuda_failed(e);
    // the three tile kernels run if the check left 0 in the gate, the general kernels behind them if it left 1
    // profile events: the whole backward (either route) lies between the backward's start and stop events; the
    // gated general kernels behind the tile kernels do not move them
    e = record(2, st);
    if (e != cudaSuccess) return cuda_failed(e);
    const bool tiled = dsa3d::try_bounded_offsets_backward(q, k, v, offsets, lse, dout, dq, dk, dv, doffsets, workspace, gate,
                                                          pr, st, &e);
    if (tiled && e != cudaSuccess) return cuda_failed(e);
    if (!tiled)
        return dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets, workspace,
                                    workspace_bytes, dtype, stream, true);
    cudaEvent_t held[6];
    for (int i = 0; i < 6; ++i) { held[i] = g_events[i]; g_events[i] = nullptr; }
    const int rc2 = dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets, workspace,
                                         workspace_bytes, dtype, stream, true, gate);
    for (int i = 0; i < 6; ++i) g_events[i] = held[i];
    if (rc2 != DSA3D_OK) return rc2;
    e = record(3, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

size_t dsa3d_backward_fixed_window_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3],
                                                   int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    // two fp32 coefficients per sample, then (where the tensor-core table kernel covers the shape)
    // the dot-product tables of every query's box
    const size_t coef = (static_cast<size_t>(pr.items) * pr.P * sizeof(float2) + 255) & ~static_cast<size_t>(255);
    const size_t table = static_cast<size_t>(pr.items) * dsa3d::fixed_window_table_floats(pr, dtype == DSA3D_BF16) * sizeof(float);
    return coef + table;
}

int dsa3d_backward_fixed_window(const void* q, const void* k, const void* v, const float* lse, const void* dout, int T,
                                int H, int W, int heads, int d, const int window[3], void* dq, void* dk, void* dv,
                                float* doffsets, void* workspace, size_t workspace_bytes, int dtype, void* stream) {
    if (!q || !k || !v || !lse || !dout || !dq || !dk || !dv) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(lse) || !aligned16(dout) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || (doffsets && !aligned16(doffsets)))
        return DSA3D_ERR_MISALIGNED;
    const size_t need = dsa3d_backward_fixed_window_workspace_bytes(T, H, W, heads, d, window, dtype);
    if (!workspace || workspace_bytes < need) return DSA3D_ERR_WORKSPACE;
    if (!aligned16(workspace)) return DSA3D_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = record(2, st);
    if (e != cudaSuccess) return cuda_failed(e);
    const float* table = nullptr;
    if (dsa3d::fixed_window_table_floats(pr, dtype == DSA3D_BF16) > 0 && !std::getenv("DSA3D_NO_TENSOR_FIXED_WINDOW")) {
        const size_t coef_bytes = (static_cast<size_t>(pr.items) * pr.P * sizeof(float2) + 255) & ~static_cast<size_t>(255);
        float* tab = reinterpret_cast<float*>(static_cast<char*>(workspace) + coef_bytes);
        if (dsa3d::try_fixed_window_tables(q, k, v, dout, tab, pr, st, &e)) {
            if (e != cudaSuccess) return cuda_failed(e);
            table = tab;
        }
    }
    e = dsa3d::launch_fixed_window_backward(q, k, v, lse, dout, dq, dk, dv, doffsets, static_cast<float2*>(workspace), table,
                                            pr, dtype == DSA3D_BF16, !std::getenv("DSA3D_NO_TENSOR_FIXED_WINDOW"), st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(3, st);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

int dsa3d_forward_residual(const void* q, const void* k, const void* v, const float* offsets, const void* residual,
                           int T, int H, int W, int heads, int d, const int window[3], void* out, float* lse,
                           int dtype, void* stream) {
    if (!residual) return DSA3D_ERR_NULL_POINTER;
    return forward_entry(q, k, v, offsets, residual, T, H, W, heads, d, window, out, lse, dtype, stream);
}

size_t dsa3d_backward_workspace_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    if (dtype == DSA3D_BF16) set_tiling(pr);
    return backward_workspace(pr, dtype, true).total;
}

int dsa3d_backward(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                   const void* dout, int T, int H, int W, int heads, int d, const int window[3], void* dq,
                   void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes, int dtype,
                   void* stream) {
    return dsa3d::backward_impl(q, k, v, offsets, lse, dout, T, H, W, heads, d, window, dq, dk, dv, doffsets,
                                workspace, workspace_bytes, dtype, stream, true);
}

}  // extern "C"

namespace {

// Everything dsa3d_backward derives from its arguments before it launches anything.
struct BackwardPlan {
    dsa3d::Problem pr;
    bool bf16 = false;
    BackwardWorkspace ws{};
    size_t count = 0;                 // elements of dk (= of dv)
    float* acc_dk = nullptr;          // fp32 accumulators (the outputs themselves for fp32 storage)
    float* acc_dv = nullptr;
    float2* coef = nullptr;
    void* scratch = nullptr;
    void* workspace = nullptr;
    int ctas = 0;                     // resident CTAs of the tile kernel
};

int backward_plan(int T, int H, int W, int heads, int d, const int* window, int dtype, bool tiled, void* dk,
                  void* dv, void* workspace, size_t workspace_bytes, BackwardPlan& plan) {
    const int rc = make_problem(T, H, W, heads, d, window, dtype, plan.pr);
    if (rc != DSA3D_OK) return rc;
    plan.bf16 = dtype == DSA3D_BF16;
    if (plan.bf16 && tiled) set_tiling(plan.pr);
    plan.ws = backward_workspace(plan.pr, dtype, tiled);
    if (plan.ws.total > 0) {
        if (!workspace || workspace_bytes < plan.ws.total) return DSA3D_ERR_WORKSPACE;
        if (!aligned16(workspace)) return DSA3D_ERR_MISALIGNED;
    }
    plan.count = static_cast<size_t>(plan.pr.items) * plan.pr.d;
    char* wsp = static_cast<char*>(workspace);
    plan.workspace = workspace;
    plan.acc_dk = plan.bf16 ? reinterpret_cast<float*>(wsp) : static_cast<float*>(dk);
    plan.acc_dv = plan.bf16 ? reinterpret_cast<float*>(wsp) + plan.count : static_cast<float*>(dv);
    plan.coef = plan.ws.coef_bytes ? reinterpret_cast<float2*>(wsp + plan.ws.acc_bytes) : nullptr;
    plan.scratch = plan.ws.scratch_bytes ? wsp + plan.ws.acc_bytes + plan.ws.coef_bytes : nullptr;
    if (plan.pr.key_blocks) {
        const dsa3d::KeyBlockLayout kb = dsa3d::key_block_layout(plan.pr);
        plan.pr.blk_count = static_cast<uint32_t*>(plan.scratch);
        plan.pr.blk_list = reinterpret_cast<uint32_t*>(static_cast<char*>(plan.scratch) + kb.count_bytes);
        plan.pr.blk_cap = kb.cap;
    }
    if (plan.coef) {
        int dev = 0, sms = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_failed(e);
        plan.ctas = sms * (dsa3d::tile_smem_bytes(plan.pr) <= 110 * 1024 ? 2 : 1);
        if (plan.ctas > kTileSlots) plan.ctas = kTileSlots;
    }
    return DSA3D_OK;
}

// Zero the dK/dV accumulators.
int backward_clear(const BackwardPlan& plan, cudaStream_t stream) {
    cudaError_t e;
    if (plan.bf16) {
        e = plan.pr.gate ? dsa3d::launch_gated_clear(plan.workspace, plan.ws.acc_bytes, plan.pr.gate, stream)
                         : cudaMemsetAsync(plan.workspace, 0, plan.ws.acc_bytes, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    } else {
        e = cudaMemsetAsync(plan.acc_dk, 0, plan.count * sizeof(float), stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = cudaMemsetAsync(plan.acc_dv, 0, plan.count * sizeof(float), stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return DSA3D_OK;
}

// The query tokens of frames [f0, f1) as a launch of their own.  With tiling on, f0 must be a
// multiple of the tile's frame count (f1 too unless it is T).
dsa3d::Problem frames_of(const dsa3d::Problem& pr, int f0, int f1) {
    dsa3d::Problem s = pr;
    const long long per_frame = static_cast<long long>(pr.H) * pr.W;
    s.q_begin = f0 * per_frame;
    s.q_count = (f1 - f0) * per_frame;
    s.items = s.q_count * pr.heads;
    if (pr.tile_t >= 1) {
        s.tt_begin = f0 / pr.tile_t;
        s.tt_count = (f1 + pr.tile_t - 1) / pr.tile_t - s.tt_begin;
    }
    return s;
}

// dQ, dOffsets of the queries of frames [f0, f1) and their contributions to dK/dV.
int backward_frames(const BackwardPlan& plan, const void* q, const void* k, const void* v, const float* offsets,
                    const float* lse, const void* dout, void* dq, float* doffsets, int f0, int f1,
                    cudaStream_t stream, cudaEvent_t after_gather) {
    const dsa3d::Problem pr = frames_of(plan.pr, f0, f1);
    cudaError_t e = record(2, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    if (pr.key_blocks) {                 // the sample lists of the key blocks start empty for every launch
        e = cudaMemsetAsync(pr.blk_count, 0, dsa3d::key_block_layout(pr).count_bytes, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    e = dsa3d::launch_backward(q, k, v, offsets, lse, dout, dq, plan.acc_dk, plan.acc_dv, doffsets, plan.coef, pr,
                               plan.bf16, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(3, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    if (after_gather) {
        e = cudaEventRecord(after_gather, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    if (plan.coef) {
        e = record(4, stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = pr.key_blocks ? dsa3d::launch_dkdv_blocks(q, dout, offsets, plan.coef, plan.acc_dk, plan.acc_dv, pr, stream)
                          : dsa3d::launch_scatter_tiles(q, dout, offsets, plan.coef, plan.acc_dk, plan.acc_dv, plan.scratch,
                                                        plan.ctas, plan.ws.entries_per_cta, pr, stream);
        if (e != cudaSuccess) return cuda_failed(e);
        e = record(5, stream);
        if (e != cudaSuccess) return cuda_failed(e);
    }
    return DSA3D_OK;
}

// Accumulators -> dk, dv (bf16 storage only; fp32 storage accumulated in place).
int backward_finish(const BackwardPlan& plan, void* dk, void* dv, cudaStream_t stream) {
    if (!plan.bf16) return DSA3D_OK;
    cudaError_t e = dsa3d::launch_convert_bf16(plan.acc_dk, dk, static_cast<long long>(plan.count), stream, plan.pr.gate);
    if (e != cudaSuccess) return cuda_failed(e);
    e = dsa3d::launch_convert_bf16(plan.acc_dv, dv, static_cast<long long>(plan.count), stream, plan.pr.gate);
    if (e != cudaSuccess) return cuda_failed(e);
    return DSA3D_OK;
}

int forward_frames(const dsa3d::Problem& full, const void* q, const void* k, const void* v, const float* offsets,
                   void* out, float* lse, bool bf16, int f0, int f1, cudaStream_t stream) {
    const dsa3d::Problem pr = frames_of(full, f0, f1);
    cudaError_t e = record(0, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    e = dsa3d::launch_forward(q, k, v, offsets, nullptr, out, lse, pr, bf16, stream);
    if (e != cudaSuccess) return cuda_failed(e);
    e = record(1, stream);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

}  // namespace

int dsa3d::backward_impl(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                         const void* dout, int T, int H, int W, int heads, int d, const int window[3],
                         void* dq, void* dk, void* dv, float* doffsets, void* workspace,
                         size_t workspace_bytes, int dtype, void* stream_, bool tiled, const int* gate) {
    if (!q || !k || !v || !offsets || !lse || !dout || !dq || !dk || !dv || !doffsets)
        return DSA3D_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(offsets) || !aligned16(lse) ||
        !aligned16(dout) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(doffsets))
        return DSA3D_ERR_MISALIGNED;
    BackwardPlan plan;
    int rc = backward_plan(T, H, W, heads, d, window, dtype, tiled, dk, dv, workspace, workspace_bytes, plan);
    if (rc != DSA3D_OK) return rc;
    plan.pr.gate = gate;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    rc = backward_clear(plan, stream);
    if (rc != DSA3D_OK) return rc;
    rc = backward_frames(plan, q, k, v, offsets, lse, dout, dq, doffsets, 0, T, stream, nullptr);
    if (rc != DSA3D_OK) return rc;
    return backward_finish(plan, dk, dv, stream);
}

extern "C" {

namespace {

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Layout of the device arena of dsa3d_step_host: offsets of each buffer, total in `total`.
struct Arena {
    size_t q, k, v, k2, v2, dout, out, dq, dk, dv, offsets, doffsets, lse, workspace, total;
    size_t row_bytes, off_bytes, lse_bytes, ws_bytes;
};

Arena arena_layout(const dsa3d::Problem& pr, int dtype) {
    Arena a;
    const size_t elt = dtype == DSA3D_BF16 ? 2 : 4;
    a.row_bytes = static_cast<size_t>(pr.items) * pr.d * elt;
    a.off_bytes = static_cast<size_t>(pr.items) * pr.P * 3 * sizeof(float);
    a.lse_bytes = static_cast<size_t>(pr.items) * sizeof(float);
    {
        dsa3d::Problem tiled = pr;
        if (dtype == DSA3D_BF16) set_tiling(tiled);
        a.ws_bytes = backward_workspace(tiled, dtype, true).total;
    }
    size_t at = 0;
    // K and V twice: the pipelined step uploads the next call's K/V while this call's kernels read theirs
    size_t* rows[10] = {&a.q, &a.k, &a.v, &a.k2, &a.v2, &a.dout, &a.out, &a.dq, &a.dk, &a.dv};
    for (size_t* r : rows) { *r = at; at += round256(a.row_bytes); }
    a.offsets = at; at += round256(a.off_bytes);
    a.doffsets = at; at += round256(a.off_bytes);
    a.lse = at; at += round256(a.lse_bytes);
    a.workspace = at; at += round256(a.ws_bytes);
    a.total = at;
    return a;
}

// Two side streams and the events of the copy/compute pipeline of dsa3d_step_host, per
// (thread, device); created on first use and kept for the life of the thread.
constexpr int kMaxSlabs = 8;
struct HostStep {
    int device = -1;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, kv_ready = nullptr, out_done = nullptr;
    cudaEvent_t q_ready[kMaxSlabs] = {}, dout_ready[kMaxSlabs] = {}, fwd_done[kMaxSlabs] = {},
                gather_done[kMaxSlabs] = {};
    // ordering between one call and the next (a wait on an event never recorded is a no-op):
    cudaEvent_t kv_free[2] = {};               // main: last kernel that reads K/V buffer b has run
    cudaEvent_t slab_in_free[kMaxSlabs] = {};  // main: q/offsets/dout of slab s consumed
    cudaEvent_t slab_dl_done[kMaxSlabs] = {};  // out: out/lse/dq/doffsets of slab s are on the host
    cudaEvent_t finish_done = nullptr;         // main: dk/dv final on the device
    cudaEvent_t dkdv_dl_done = nullptr;        // out: dk/dv are on the host
    cudaEvent_t main_done = nullptr;           // main: end of the call's kernels
    int kv_index = 0;                          // K/V buffer of the next call
    const void* last_arena = nullptr;
    long long last_shape[7] = {0, 0, 0, 0, 0, 0, 0};
};
thread_local HostStep g_host_step[8];

HostStep* host_step_resources() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    HostStep* slot = nullptr;
    for (HostStep& h : g_host_step) {
        if (h.device == dev) return &h;
        if (!slot && h.device < 0) slot = &h;
    }
    if (!slot) return nullptr;                          // more than 8 devices used from one thread
    if (cudaStreamCreateWithFlags(&slot->in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&slot->out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    cudaEvent_t* single[8] = {&slot->start, &slot->kv_ready, &slot->out_done, &slot->finish_done, &slot->dkdv_dl_done,
                              &slot->main_done, &slot->kv_free[0], &slot->kv_free[1]};
    for (cudaEvent_t* ev : single)
        if (cudaEventCreateWithFlags(ev, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    cudaEvent_t* per_slab[6] = {slot->q_ready, slot->dout_ready, slot->fwd_done, slot->gather_done, slot->slab_in_free,
                                slot->slab_dl_done};
    for (cudaEvent_t* arr : per_slab)
        for (int i = 0; i < kMaxSlabs; ++i)
            if (cudaEventCreateWithFlags(&arr[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    slot->device = dev;
    return slot;
}

}  // namespace

size_t dsa3d_step_host_arena_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    return arena_layout(pr, dtype).total;
}

namespace {

// One step enqueued on `stream_` and the two side streams.  ordered_start: uploads wait for the
// work already on the stream (the plain entry point); otherwise only for the buffers they
// overwrite, so that they overlap the previous call's kernels (the pipelined entry point).
int step_host_body(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                   const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                   void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                   void* arena, size_t arena_bytes, int dtype, void* stream_, bool ordered_start) {
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
    HostStep* hs = host_step_resources();
    if (!hs) return cuda_failed(cudaGetLastError());     // side streams / events could not be created
    cudaError_t e;
#define DSA3D_TRY(call)                         \
    do {                                        \
        e = (call);                             \
        if (e != cudaSuccess) return cuda_failed(e); \
    } while (0)
    // The query side of the step (q, offsets, dout in; out, lse, dq, doffsets back) is cut
    // into slabs of whole frames.  Side stream `in` uploads K and V, then slab after slab;
    // the main stream runs the forward and the backward of a slab as soon as its inputs are
    // there; side stream `out` carries each slab's results back while the next slab computes.
    // Only K/V (needed by every query) at the start and dK/dV (final after the last slab) at
    // the end are not hidden behind kernels.
    const bool bf16 = dtype == DSA3D_BF16;
    BackwardPlan plan;
    int st = backward_plan(T, H, W, heads, d, window, dtype, true, base + a.dk, base + a.dv,
                           a.ws_bytes ? base + a.workspace : nullptr, a.ws_bytes, plan);
    if (st != DSA3D_OK) return st;
    const int unit = plan.pr.tile_t >= 1 ? plan.pr.tile_t : 1;          // slabs start on tile boundaries
    int slab_frames = (T + kMaxSlabs - 1) / kMaxSlabs;
    slab_frames = (slab_frames + unit - 1) / unit * unit;
    const int slabs = (T + slab_frames - 1) / slab_frames;
    const size_t elt = bf16 ? 2 : 4;
    const size_t frame_rows = static_cast<size_t>(H) * W * heads;
    const size_t frame_row_bytes = frame_rows * d * elt;
    const size_t frame_off_bytes = frame_rows * pr.P * 3 * sizeof(float);
    const size_t frame_lse_bytes = frame_rows * sizeof(float);
    const char* q_hb = static_cast<const char*>(q_h);
    const char* off_hb = reinterpret_cast<const char*>(offsets_h);
    const char* dout_hb = static_cast<const char*>(dout_h);

    // A call with another arena or shape than the previous one shares no per-slab ordering with
    // it: wait for all of the previous call first.
    const long long shape[7] = {T, H, W, heads, d, dtype, static_cast<long long>(window[0]) * 10000 + window[1] * 100 + window[2]};
    bool same = hs->last_arena == arena;
    for (int i = 0; i < 7; ++i) same = same && hs->last_shape[i] == shape[i];
    if (!same) {
        DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->main_done, 0));
        DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->out_done, 0));
        DSA3D_TRY(cudaStreamWaitEvent(stream, hs->out_done, 0));
        hs->last_arena = arena;
        for (int i = 0; i < 7; ++i) hs->last_shape[i] = shape[i];
    }
    // the previous call's kernels come first even if it was queued on another stream (they share the
    // workspace and the result buffers; on the same stream this wait is already satisfied)
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->main_done, 0));
    if (ordered_start) {
        DSA3D_TRY(cudaEventRecord(hs->start, stream));
        DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->start, 0));
        DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->start, 0));
    }
    const int kvb = hs->kv_index;
    hs->kv_index ^= 1;
    char* k_d = base + (kvb ? a.k2 : a.k);
    char* v_d = base + (kvb ? a.v2 : a.v);
    DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->kv_free[kvb], 0));
    DSA3D_TRY(cudaMemcpyAsync(k_d, k_h, a.row_bytes, cudaMemcpyHostToDevice, hs->in));
    DSA3D_TRY(cudaMemcpyAsync(v_d, v_h, a.row_bytes, cudaMemcpyHostToDevice, hs->in));
    DSA3D_TRY(cudaEventRecord(hs->kv_ready, hs->in));
    for (int s = 0; s < slabs; ++s) {
        const int f0 = s * slab_frames, f1 = f0 + slab_frames < T ? f0 + slab_frames : T;
        const size_t nf = static_cast<size_t>(f1 - f0);
        DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->slab_in_free[s], 0));     // the previous call's use of this slab
        DSA3D_TRY(cudaMemcpyAsync(base + a.q + f0 * frame_row_bytes, q_hb + f0 * frame_row_bytes,
                                  nf * frame_row_bytes, cudaMemcpyHostToDevice, hs->in));
        DSA3D_TRY(cudaMemcpyAsync(base + a.offsets + f0 * frame_off_bytes, off_hb + f0 * frame_off_bytes,
                                  nf * frame_off_bytes, cudaMemcpyHostToDevice, hs->in));
        DSA3D_TRY(cudaEventRecord(hs->q_ready[s], hs->in));
        DSA3D_TRY(cudaMemcpyAsync(base + a.dout + f0 * frame_row_bytes, dout_hb + f0 * frame_row_bytes,
                                  nf * frame_row_bytes, cudaMemcpyHostToDevice, hs->in));
        DSA3D_TRY(cudaEventRecord(hs->dout_ready[s], hs->in));
    }

    // fp32 storage accumulates dk/dv in place: the previous call's download of them comes first.
    // (bf16 accumulates in the workspace; its dk/dv are only written by backward_finish below.)
    if (!bf16) DSA3D_TRY(cudaStreamWaitEvent(stream, hs->dkdv_dl_done, 0));
    st = backward_clear(plan, stream);
    if (st != DSA3D_OK) return st;
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->kv_ready, 0));
    const float* off_d = reinterpret_cast<const float*>(base + a.offsets);
    float* lse_d = reinterpret_cast<float*>(base + a.lse);
    float* doff_d = reinterpret_cast<float*>(base + a.doffsets);
    for (int s = 0; s < slabs; ++s) {
        const int f0 = s * slab_frames, f1 = f0 + slab_frames < T ? f0 + slab_frames : T;
        const size_t nf = static_cast<size_t>(f1 - f0);
        DSA3D_TRY(cudaStreamWaitEvent(stream, hs->q_ready[s], 0));
        DSA3D_TRY(cudaStreamWaitEvent(stream, hs->slab_dl_done[s], 0));     // the previous call's results of this slab
        st = forward_frames(pr, base + a.q, k_d, v_d, off_d, base + a.out, lse_d, bf16, f0, f1, stream);
        if (st != DSA3D_OK) return st;
        DSA3D_TRY(cudaEventRecord(hs->fwd_done[s], stream));
        DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->fwd_done[s], 0));
        DSA3D_TRY(cudaMemcpyAsync(static_cast<char*>(out_h) + f0 * frame_row_bytes,
                                  base + a.out + f0 * frame_row_bytes, nf * frame_row_bytes,
                                  cudaMemcpyDeviceToHost, hs->out));
        DSA3D_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(lse_h) + f0 * frame_lse_bytes,
                                  base + a.lse + f0 * frame_lse_bytes, nf * frame_lse_bytes,
                                  cudaMemcpyDeviceToHost, hs->out));

        DSA3D_TRY(cudaStreamWaitEvent(stream, hs->dout_ready[s], 0));
        st = backward_frames(plan, base + a.q, k_d, v_d, off_d, lse_d, base + a.dout, base + a.dq,
                             doff_d, f0, f1, stream, hs->gather_done[s]);
        if (st != DSA3D_OK) return st;
        DSA3D_TRY(cudaEventRecord(hs->slab_in_free[s], stream));
        DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->gather_done[s], 0));
        DSA3D_TRY(cudaMemcpyAsync(static_cast<char*>(dq_h) + f0 * frame_row_bytes,
                                  base + a.dq + f0 * frame_row_bytes, nf * frame_row_bytes,
                                  cudaMemcpyDeviceToHost, hs->out));
        DSA3D_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(doffsets_h) + f0 * frame_off_bytes,
                                  base + a.doffsets + f0 * frame_off_bytes, nf * frame_off_bytes,
                                  cudaMemcpyDeviceToHost, hs->out));
        DSA3D_TRY(cudaEventRecord(hs->slab_dl_done[s], hs->out));
    }
    DSA3D_TRY(cudaEventRecord(hs->kv_free[kvb], stream));                 // no later kernel of this call reads K/V
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->dkdv_dl_done, 0));          // the previous call's dk/dv are on the host
    st = backward_finish(plan, base + a.dk, base + a.dv, stream);
    if (st != DSA3D_OK) return st;
    DSA3D_TRY(cudaEventRecord(hs->finish_done, stream));
    DSA3D_TRY(cudaEventRecord(hs->main_done, stream));
    DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->finish_done, 0));
    DSA3D_TRY(cudaMemcpyAsync(dk_h, base + a.dk, a.row_bytes, cudaMemcpyDeviceToHost, hs->out));
    DSA3D_TRY(cudaMemcpyAsync(dv_h, base + a.dv, a.row_bytes, cudaMemcpyDeviceToHost, hs->out));
    DSA3D_TRY(cudaEventRecord(hs->dkdv_dl_done, hs->out));
    DSA3D_TRY(cudaEventRecord(hs->out_done, hs->out));
#undef DSA3D_TRY
    return DSA3D_OK;
}

}  // namespace

int dsa3d_step_host(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                    const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                    void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                    void* arena, size_t arena_bytes, int dtype, void* stream) {
    const int rc = step_host_body(q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window, out_h, lse_h, dq_h, dk_h,
                                  dv_h, doffsets_h, arena, arena_bytes, dtype, stream, true);
    if (rc != DSA3D_OK) return rc;
    return dsa3d_step_host_flush(stream);                        // the step is over when `stream` is
}

int dsa3d_step_host_pipelined(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h,
                              const void* dout_h, int T, int H, int W, int heads, int d, const int window[3],
                              void* out_h, float* lse_h, void* dq_h, void* dk_h, void* dv_h, float* doffsets_h,
                              void* arena, size_t arena_bytes, int dtype, void* stream) {
    return step_host_body(q_h, k_h, v_h, offsets_h, dout_h, T, H, W, heads, d, window, out_h, lse_h, dq_h, dk_h, dv_h,
                          doffsets_h, arena, arena_bytes, dtype, stream, false);
}

int dsa3d_step_host_flush(void* stream) {
    HostStep* hs = host_step_resources();
    if (!hs) return cuda_failed(cudaGetLastError());
    const cudaError_t e = cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), hs->out_done, 0);
    return e == cudaSuccess ? DSA3D_OK : cuda_failed(e);
}

// Forward only on host buffers (inference / sampling): device arena = q, k, v, out rows,
// offsets, lse.
size_t dsa3d_forward_host_arena_bytes(int T, int H, int W, int heads, int d, const int window[3], int dtype) {
    dsa3d::Problem pr;
    if (make_problem(T, H, W, heads, d, window, dtype, pr) != DSA3D_OK) return 0;
    const size_t elt = dtype == DSA3D_BF16 ? 2 : 4;
    const size_t rows = round256(static_cast<size_t>(pr.items) * pr.d * elt);
    return 4 * rows + round256(static_cast<size_t>(pr.items) * pr.P * 3 * sizeof(float)) +
           round256(static_cast<size_t>(pr.items) * sizeof(float));
}

int dsa3d_forward_host(const void* q_h, const void* k_h, const void* v_h, const float* offsets_h, int T, int H, int W,
                       int heads, int d, const int window[3], void* out_h, float* lse_h, void* arena,
                       size_t arena_bytes, int dtype, void* stream_) {
    if (!q_h || !k_h || !v_h || !offsets_h || !out_h || !lse_h || !arena) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return DSA3D_ERR_MISALIGNED;
    if (arena_bytes < dsa3d_forward_host_arena_bytes(T, H, W, heads, d, window, dtype)) return DSA3D_ERR_WORKSPACE;
    const bool bf16 = dtype == DSA3D_BF16;
    const size_t elt = bf16 ? 2 : 4;
    const size_t row_bytes = static_cast<size_t>(pr.items) * pr.d * elt;
    const size_t rows = round256(row_bytes);
    char* base = static_cast<char*>(arena);
    char *q_d = base, *k_d = base + rows, *v_d = base + 2 * rows, *out_d = base + 3 * rows;
    char* off_d = base + 4 * rows;
    char* lse_d = off_d + round256(static_cast<size_t>(pr.items) * pr.P * 3 * sizeof(float));
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    HostStep* hs = host_step_resources();
    if (!hs) return cuda_failed(cudaGetLastError());
    cudaError_t e;
#define DSA3D_TRY(call)                         \
    do {                                        \
        e = (call);                             \
        if (e != cudaSuccess) return cuda_failed(e); \
    } while (0)
    // K and V first (every query needs all of them), then slabs of frames: a slab's q and offsets
    // go up on one side stream while earlier slabs compute, its out and lse come back on the other.
    int slab_frames = (T + kMaxSlabs - 1) / kMaxSlabs;
    const int slabs = (T + slab_frames - 1) / slab_frames;
    const size_t frame_rows = static_cast<size_t>(H) * W * heads;
    const size_t frame_row_bytes = frame_rows * d * elt;
    const size_t frame_off_bytes = frame_rows * pr.P * 3 * sizeof(float);
    const size_t frame_lse_bytes = frame_rows * sizeof(float);
    // transfers that pipelined steps may still have in flight on the side streams come first
    // (this call may reuse their arena), and a later step shares no per-slab ordering with it
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->out_done, 0));
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->main_done, 0));      // their kernels too, if queued on another stream
    hs->last_arena = nullptr;
    DSA3D_TRY(cudaEventRecord(hs->start, stream));
    DSA3D_TRY(cudaStreamWaitEvent(hs->in, hs->start, 0));
    DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->start, 0));
    DSA3D_TRY(cudaMemcpyAsync(k_d, k_h, row_bytes, cudaMemcpyHostToDevice, hs->in));
    DSA3D_TRY(cudaMemcpyAsync(v_d, v_h, row_bytes, cudaMemcpyHostToDevice, hs->in));
    DSA3D_TRY(cudaEventRecord(hs->kv_ready, hs->in));
    for (int s = 0; s < slabs; ++s) {
        const int f0 = s * slab_frames, f1 = f0 + slab_frames < T ? f0 + slab_frames : T;
        const size_t nf = static_cast<size_t>(f1 - f0);
        DSA3D_TRY(cudaMemcpyAsync(q_d + f0 * frame_row_bytes, static_cast<const char*>(q_h) + f0 * frame_row_bytes,
                                  nf * frame_row_bytes, cudaMemcpyHostToDevice, hs->in));
        DSA3D_TRY(cudaMemcpyAsync(off_d + f0 * frame_off_bytes,
                                  reinterpret_cast<const char*>(offsets_h) + f0 * frame_off_bytes, nf * frame_off_bytes,
                                  cudaMemcpyHostToDevice, hs->in));
        DSA3D_TRY(cudaEventRecord(hs->q_ready[s], hs->in));
    }
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->kv_ready, 0));
    for (int s = 0; s < slabs; ++s) {
        const int f0 = s * slab_frames, f1 = f0 + slab_frames < T ? f0 + slab_frames : T;
        const size_t nf = static_cast<size_t>(f1 - f0);
        DSA3D_TRY(cudaStreamWaitEvent(stream, hs->q_ready[s], 0));
        const int st = forward_frames(pr, q_d, k_d, v_d, reinterpret_cast<const float*>(off_d), out_d,
                                      reinterpret_cast<float*>(lse_d), bf16, f0, f1, stream);
        if (st != DSA3D_OK) return st;
        DSA3D_TRY(cudaEventRecord(hs->fwd_done[s], stream));
        DSA3D_TRY(cudaStreamWaitEvent(hs->out, hs->fwd_done[s], 0));
        DSA3D_TRY(cudaMemcpyAsync(static_cast<char*>(out_h) + f0 * frame_row_bytes, out_d + f0 * frame_row_bytes,
                                  nf * frame_row_bytes, cudaMemcpyDeviceToHost, hs->out));
        DSA3D_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(lse_h) + f0 * frame_lse_bytes, lse_d + f0 * frame_lse_bytes,
                                  nf * frame_lse_bytes, cudaMemcpyDeviceToHost, hs->out));
    }
    DSA3D_TRY(cudaEventRecord(hs->out_done, hs->out));
    DSA3D_TRY(cudaStreamWaitEvent(stream, hs->out_done, 0));     // the call is over when `stream` is
#undef DSA3D_TRY
    return DSA3D_OK;
}

int dsa3d_set_profile_events(void* fwd_start, void* fwd_stop, void* bwd_start, void* bwd_stop,
                             void* scatter_start, void* scatter_stop) {
    g_events[0] = static_cast<cudaEvent_t>(fwd_start);
    g_events[1] = static_cast<cudaEvent_t>(fwd_stop);
    g_events[2] = static_cast<cudaEvent_t>(bwd_start);
    g_events[3] = static_cast<cudaEvent_t>(bwd_stop);
    g_events[4] = static_cast<cudaEvent_t>(scatter_start);
    g_events[5] = static_cast<cudaEvent_t>(scatter_stop);
    return DSA3D_OK;
}

// A batch is `batch` independent videos stored back to back; each one is a problem of its
// own (no sample of one video ever reads another), so the batched entry points run the
// single-video kernels once per video on the same stream, reusing one workspace.
int dsa3d_forward_batch(const void* q, const void* k, const void* v, const float* offsets, int batch, int T,
                        int H, int W, int heads, int d, const int window[3], void* out, float* lse, int dtype,
                        void* stream) {
    if (batch < 1) return DSA3D_ERR_BAD_SHAPE;
    if (!q || !k || !v || !offsets || !out || !lse) return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    const size_t rows = static_cast<size_t>(pr.items) * pr.d * (dtype == DSA3D_BF16 ? 2 : 4);
    const size_t offs = static_cast<size_t>(pr.items) * pr.P * 3;
    for (int b = 0; b < batch; ++b) {
        const int st = dsa3d_forward(static_cast<const char*>(q) + b * rows, static_cast<const char*>(k) + b * rows,
                                     static_cast<const char*>(v) + b * rows, offsets + b * offs, T, H, W, heads, d,
                                     window, static_cast<char*>(out) + b * rows, lse + b * static_cast<size_t>(pr.items),
                                     dtype, stream);
        if (st != DSA3D_OK) return st;
    }
    return DSA3D_OK;
}

int dsa3d_backward_batch(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                         const void* dout, int batch, int T, int H, int W, int heads, int d, const int window[3],
                         void* dq, void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes,
                         int dtype, void* stream) {
    if (batch < 1) return DSA3D_ERR_BAD_SHAPE;
    if (!q || !k || !v || !offsets || !lse || !dout || !dq || !dk || !dv || !doffsets)
        return DSA3D_ERR_NULL_POINTER;
    dsa3d::Problem pr;
    const int rc = make_problem(T, H, W, heads, d, window, dtype, pr);
    if (rc != DSA3D_OK) return rc;
    const size_t rows = static_cast<size_t>(pr.items) * pr.d * (dtype == DSA3D_BF16 ? 2 : 4);
    const size_t offs = static_cast<size_t>(pr.items) * pr.P * 3;
    for (int b = 0; b < batch; ++b) {
        const int st = dsa3d_backward(
            static_cast<const char*>(q) + b * rows, static_cast<const char*>(k) + b * rows,
            static_cast<const char*>(v) + b * rows, offsets + b * offs, lse + b * static_cast<size_t>(pr.items),
            static_cast<const char*>(dout) + b * rows, T, H, W, heads, d, window, static_cast<char*>(dq) + b * rows,
            static_cast<char*>(dk) + b * rows, static_cast<char*>(dv) + b * rows, doffsets + b * offs, workspace,
            workspace_bytes, dtype, stream);
        if (st != DSA3D_OK) return st;
    }
    return DSA3D_OK;
}

int dsa3d_debug_build(void) {
#ifdef DSA3D_DEBUG
    return 1;
#else
    return 0;
#endif
}

int dsa3d_debug_first_violation(int* code, long long* offset) {
    if (!code || !offset) return DSA3D_ERR_NULL_POINTER;
    *code = 0;
    *offset = 0;
#ifdef DSA3D_DEBUG
    unsigned long long word = 0ull;
    const cudaError_t e = cudaMemcpyFromSymbol(&word, g_debug_word, sizeof(word));     // synchronises with the device
    if (e != cudaSuccess) return cuda_failed(e);
    *code = static_cast<int>(word >> 56);
    long long off = static_cast<long long>(word & ((1ull << 56) - 1));
    if (off & (1LL << 55)) off -= (1LL << 56);                                          // sign of the 56-bit field
    *offset = off;
#endif
    return DSA3D_OK;
}

int dsa3d_debug_clear(void) {
#ifdef DSA3D_DEBUG
    const unsigned long long zero = 0ull;
    const cudaError_t e = cudaMemcpyToSymbol(g_debug_word, &zero, sizeof(zero));
    if (e != cudaSuccess) return cuda_failed(e);
#endif
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
        case DSA3D_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        default: return "unknown status";
    }
}

int dsa3d_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
