// Internal launch interface between the C-ABI layer and the kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>

#include "dsa3d_common.cuh"

namespace dsa3d {

// `addend` (same layout and type as out, or NULL) is added to the attention output before the
// single rounding to the storage type: the first term of Eq. 1.
// `gate` (or NULL): a device word; when given, the kernel does nothing unless it is non-zero.
cudaError_t launch_forward(const void* q, const void* k, const void* v, const float* offsets, const void* addend,
                           void* out, float* lse, const Problem& pr, bool bf16, cudaStream_t stream,
                           const int* gate = nullptr);

// Remember `e` as the calling thread's last CUDA error (dsa3d_last_cuda_error) and return
// DSA3D_ERR_CUDA.
int note_cuda_error(cudaError_t e);

// acc_dk / acc_dv: fp32 accumulators [N, heads, d], zeroed by the caller.  For fp32 storage
// they are the dk / dv outputs themselves.  coef [N*heads, P] receives the two scatter
// coefficients of every sample when the problem is tiled (pr.tile_t >= 1), else it may be
// NULL.  Corners inside the halo of their query's tile are left to launch_scatter_tiles.
cudaError_t launch_backward(const void* q, const void* k, const void* v, const float* offsets,
                            const float* lse, const void* dout, void* dq, float* acc_dk, float* acc_dv,
                            float* doffsets, float2* coef, const Problem& pr, bool bf16, cudaStream_t stream);

// bf16 storage only: the in-halo part of the dK/dV scatter, pre-reduced per query tile.
// `scratch` holds `ctas` regions of `entries_per_cta` 8-byte entries.
cudaError_t launch_scatter_tiles(const void* q, const void* dout, const float* offsets, const float2* coef,
                                 float* acc_dk, float* acc_dv, void* scratch, int ctas,
                                 long long entries_per_cta, const Problem& pr, cudaStream_t stream);

// Dynamic shared memory of the tile kernel for this problem's tiling.
size_t tile_smem_bytes(const Problem& pr);

// dK/dV of bf16 problems by key blocks on the tensor cores (dsa3d_backward_blocks.cu) instead of
// launch_scatter_tiles: adds, for the query tokens of `pr`, every contribution the gather kernel listed for a
// key block (block_lists_append, with pr.key_blocks set and the counters cleared before its launch) to the
// accumulators.  key_block_layout: sizes of the counters, the per-block lists (pr.blk_count, pr.blk_list follow
// each other in one buffer) and the sorted records of the resident CTAs behind them.
struct KeyBlockLayout { size_t count_bytes, list_bytes, sorted_bytes; int cap; long long blocks; };
KeyBlockLayout key_block_layout(const Problem& pr);
bool key_blocks_shape_covered(const Problem& pr);
cudaError_t launch_dkdv_blocks(const void* q, const void* dout, const float* offsets, const float2* coef, float* acc_dk,
                               float* acc_dv, const Problem& pr, cudaStream_t stream);

// fp32 accumulators -> bf16 outputs (round to nearest even).
cudaError_t launch_convert_bf16(const float* acc, void* dst, long long count, cudaStream_t stream,
                                const int* gate = nullptr);
// Zeroes `bytes` (a multiple of 16) at `dst` unless *gate is 0.
cudaError_t launch_gated_clear(void* dst, size_t bytes, const int* gate, cudaStream_t stream);

// Shared implementation of dsa3d_backward.  `tiled` selects the tile pre-reduction of the
// dK/dV scatter (bf16 only; needs the large workspace); without it the workspace is just the
// two fp32 accumulators.  Returns a dsa3d_status.
int backward_impl(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                  const void* dout, int T, int H, int W, int heads, int d, const int window[3], void* dq,
                  void* dk, void* dv, float* doffsets, void* workspace, size_t workspace_bytes, int dtype,
                  void* stream, bool tiled, const int* gate = nullptr);

// Backward of the fixed-window variant (dsa3d_fixed_window_backward.cu): dq, dk, dv in the storage
// type, doffsets (may be NULL), coef [N*heads, P] scratch.  `table` (or NULL): the dot products
// q.K_j and dO.V_j of every query's box as try_fixed_window_tables leaves them; the kernel then
// reads them instead of gathering K and V rows for them.  `tile_grad`: let the tile kernel of
// dsa3d_fixed_window_tile_grad.cu form dq, dk and dv where it covers the shape.
cudaError_t launch_fixed_window_backward(const void* q, const void* k, const void* v, const float* lse,
                                         const void* dout, void* dq, void* dk, void* dv, float* doffsets,
                                         float2* coef, const float* table, const Problem& pr, bool bf16,
                                         bool tile_grad, cudaStream_t stream);

// Dot-product tables of the fixed-window backward on the tensor cores (dsa3d_fixed_window_tables.cu).
// fixed_window_table_floats: floats per (token, head) item, 0 when the shape is not covered.
// try_fixed_window_tables: false when the shape is not covered (nothing launched).
int fixed_window_table_floats(const Problem& pr, bool bf16);

// The three weighted row sums of the fixed-window backward (dQ over the K region, dK over the q region, dV over
// the dO region) per tile of 4 x 4 x 8 outputs with the region in shared memory (dsa3d_fixed_window_tile_grad.cu),
// from the coefficient pairs the query kernel left.  covers: bf16, 64 or 128 channels, windows (3,3,3), (2,2,2).
// try_...: false when nothing was launched (shape not covered, or the tensor maps could not be made).
bool fixed_window_tile_grad_covers(const Problem& pr, bool bf16);
bool try_fixed_window_tile_grad(const void* q, const void* k, const void* dout, const float2* coef, void* dq, void* dk,
                                void* dv, const Problem& pr, cudaStream_t stream, cudaError_t* err);
bool try_bounded_offsets_planes_grad(const void* q, const void* k, const void* dout, const float* coef_planes, void* dq,
                                     void* dk, void* dv, const Problem& pr, const int* gate, cudaStream_t stream,
                                     cudaError_t* err);

// Backward for learned offsets below 1 in size, window (3,3,3) (dsa3d_bounded_offsets_backward.cu): tables,
// per-query arithmetic and the three tile sums, all doing nothing unless *gate is 0.  Returns false when
// nothing was launched (shape not covered).  `workspace`: bounded_offsets_backward_bytes(pr) bytes.
bool bounded_offsets_backward_covers(const Problem& pr, bool bf16);
size_t bounded_offsets_backward_bytes(const Problem& pr);
bool try_bounded_offsets_backward(const void* q, const void* k, const void* v, const float* offsets, const float* lse,
                                  const void* dout, void* dq, void* dk, void* dv, float* doffsets, void* workspace,
                                  const int* gate, const Problem& pr, cudaStream_t stream, cudaError_t* err);

// The dot-product tables of the box a query's samples can touch when every learned offset is below 1 in
// size (window (3,3,3): 6 x 6 x 6 positions from query - 2, dsa3d_fixed_window_tables.cu); the kernel does
// nothing unless *gate is 0.
int bounded_offsets_table_floats();
bool try_bounded_offsets_tables(const void* q, const void* k, const void* v, const void* dout, float* table,
                                const Problem& pr, const int* gate, cudaStream_t stream, cudaError_t* err);

// The same three sums for the larger windows ((3,5,5), (3,7,7); bf16, 64 or 128 channels) as products
//  C_plane . X_plane  on the tensor cores, one region plane at a time (dsa3d_fixed_window_planes_grad.cu).
bool fixed_window_planes_grad_covers(const Problem& pr, bool bf16);
// `coef_planes`: the coefficients as one plane of ck and one of cv, each [head][sample][token].
bool try_fixed_window_planes_grad(const void* q, const void* k, const void* dout, const float* coef_planes, void* dq, void* dk,
                                  void* dv, const Problem& pr, cudaStream_t stream, cudaError_t* err);
bool try_fixed_window_tables(const void* q, const void* k, const void* v, const void* dout, float* table,
                             const Problem& pr, cudaStream_t stream, cudaError_t* err);

// Host side of the TMA kernels (dsa3d_producer.cu).  encode_tensor_map_bf16: a tiled map over
// a bf16 tensor of `rank` dimensions (innermost first; strides_bytes has rank-1 entries, the
// innermost stride being 2), zero fill outside the tensor, 128-byte swizzle or none.
bool encode_tensor_map_bf16(CUtensorMap* map, const void* base, int rank, const unsigned long long* dims,
                            const unsigned long long* strides_bytes, const unsigned* box, bool swizzle128);

// Device address of the flag a tensor-core kernel raises when one of its bounded waits runs
// out (read by dsa3d_device_timeout_flag); NULL if it cannot be looked up.
int* timeout_flag_device_address();

// Fixed-window forward on the tensor cores (dsa3d_fixed_window.cu).  Returns false when the
// shape is not one it covers (the caller then uses the general kernel with zero offsets);
// *err receives a launch error.
bool try_fixed_window_forward(const void* q, const void* k, const void* v, void* out, float* lse, const Problem& pr,
                              cudaStream_t stream, cudaError_t* err);

// The same for windows (3,5,5) and (3,7,7) (dsa3d_fixed_window_planes.cu): both contractions on the
// tensor cores, the halo region taken one plane at a time.
bool try_fixed_window_forward_planes(const void* q, const void* k, const void* v, void* out, float* lse,
                                     const Problem& pr, cudaStream_t stream, cudaError_t* err);

// Forward for learned offsets below 1 in size on every axis (dsa3d_fixed_window_planes.cu): the samples of
// a query then stay inside the box "window grown by one position", and the operator runs as dense tile
// attention on the tensor cores.  launch_offsets_bound_check leaves *gate = 0 if all `count` offset
// components are finite and below 1 in size, else 1; try_bounded_offsets_forward launches the tile kernel,
// which does nothing unless *gate == 0 (false: shape not covered, nothing launched).
bool bounded_offsets_shape_covered(const Problem& pr, bool bf16);
cudaError_t launch_offsets_bound_check(const float* offsets, long long count, int* gate, cudaStream_t stream);
bool try_bounded_offsets_forward(const void* q, const void* k, const void* v, const float* offsets, const int* gate,
                                 void* out, float* lse, const Problem& pr, cudaStream_t stream, cudaError_t* err);

}  // namespace dsa3d
