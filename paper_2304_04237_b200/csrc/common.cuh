// Shared declarations of the slide-attention library: problem description, element access,
// and the launchers each kernel file exports to the API layer.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "slide_attn.h"

namespace slide_attn {

// One forward problem.  Channel c = h*head_dim + e; C = heads*head_dim; k2 = ksize*ksize.
struct Problem {
    int B, H, W, heads, head_dim, ksize;
    int has_bias;
    slide_attn_dtype dtype;
    const void* q;
    const void* k;
    const void* v;
    const float* wk;     // [C][k2 slot][k2 tap]
    const float* wv;
    const float* bias;   // [heads][k2] or nullptr
    void* out;
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// TMA tensor map of a [B][H][W][C] tensor (bf16: elem_bytes 2, fp32: 4) seen as 4-D (C, W, H, B) with
// a box of box_c channels x box_w columns x box_h rows; out-of-map elements read as zero.
bool tensor_map_available();
bool make_tile_map(CUtensorMap* map, const void* base, int elem_bytes, int B, int H, int W, int C,
                   int box_c, int box_w, int box_h);

// Launchers.  Each returns cudaGetLastError() of its launch(es).
cudaError_t launch_direct(const Problem& p, cudaStream_t stream);
bool direct_supports(int head_dim, int ksize);

// STRIP variant: generic fp32 path with transposed weights (strip_workspace_bytes, written by the
// prep launch of every forward) and four pixels per warp.
bool strip_supports(int head_dim, int ksize);
size_t strip_workspace_bytes(int heads, int head_dim, int ksize);
cudaError_t launch_strip_prep(const Problem& p, void* workspace, cudaStream_t stream);
cudaError_t launch_strip_main(const Problem& p, const void* workspace, cudaStream_t stream);

// MMA variant.  `workspace` holds the re-laid-out weights (mma_workspace_bytes), written by the
// prep launch and read by the main launch on the same stream.  mma_setup must have succeeded once
// on the device before the first main launch.
bool mma_supports(slide_attn_dtype dtype, int head_dim, int ksize);
size_t mma_workspace_bytes(int heads);
cudaError_t mma_setup();
cudaError_t launch_mma_prep(const Problem& p, void* workspace, cudaStream_t stream);
cudaError_t launch_mma_main(const Problem& p, const void* workspace, int* d_status, cudaStream_t stream);


// UMMA_TS variant: both contractions on tcgen05 with their A operands in tensor memory.  A prep launch
// writes the bf16 B images of every head (umma_ts_workspace_bytes) that the main launch's CTAs copy in.
bool umma_ts_supports(slide_attn_dtype dtype, int head_dim, int ksize);
cudaError_t umma_ts_setup();
size_t umma_ts_workspace_bytes(int heads);
cudaError_t launch_umma_ts_prep(const Problem& p, void* workspace, cudaStream_t stream);
cudaError_t launch_umma_ts(const Problem& p, const void* workspace, int* d_status, int num_sms, cudaStream_t stream);

// Fixed-shift fast path: plain k x k local attention for weights that are exactly the one-hot shift
// kernels (head_dim 32, k <= 9, fp32 or bf16).  launch_shift_check sets the status word to 2 when a
// weight differs from the one-hot kernel.
bool shift_supports(int head_dim, int ksize);
cudaError_t launch_shift_check(const Problem& p, int* d_status, cudaStream_t stream);
cudaError_t launch_shift(const Problem& p, int* d_status, cudaStream_t stream);

// Backward pass (head_dim 32, k = 1 or 3, both dtypes): gradients of the forward's inputs.
struct BackwardArgs {
    const void* dout;    // [B][H][W][heads][head_dim], the problem's dtype
    void* dq;            // same shape and dtype
    void* dk;
    void* dv;
    float* dwk;          // [C][k*k][k*k]
    float* dwv;
    float* dbias;        // [heads][k*k] or nullptr
};
bool backward_supports(int head_dim, int ksize);
size_t backward_workspace_bytes(int B, int H, int W, int heads, int ksize);
cudaError_t launch_backward(const Problem& p, const BackwardArgs& ga, const void* wt, void* ws, int* d_status,
                            int num_sms, cudaStream_t stream);

// MMA_WIDE variant: general weights with large windows on mma.sync tensor cores (bf16, head_dim 32,
// k = 3, 5, 7, 9); a prep launch writes the weights as B fragments into `workspace`.
bool mma_wide_supports(slide_attn_dtype dtype, int head_dim, int ksize);
size_t mma_wide_workspace_bytes(int heads, int ksize);
cudaError_t launch_mma_wide(const Problem& p, void* workspace, int* d_status, cudaStream_t stream);

// TILE variant: generic weights, CUDA cores, TMA-staged halo tiles (head_dim 32, k <= 9, both dtypes).
// Reads the transposed weights that launch_strip_prep writes.
bool tile_supports(int head_dim, int ksize);
cudaError_t launch_tile(const Problem& p, const void* workspace, int* d_status, cudaStream_t stream);

// Projections of a block (Eq. 1 / Eq. 3) as a tcgen05 GEMM: y[i] = x w[i] for nmat row-major fp32 [c_in][c_out]
// matrices, x and y bf16 with channels contiguous.  proj_setup must have succeeded once on the device.
bool proj_supports(int c_in, int c_out);
cudaError_t proj_setup();
cudaError_t launch_proj(const void* x, long long rows, int c_in, const float* w, int c_out, int nmat,
                        void* const* y, int* d_status, int num_sms, cudaStream_t stream);

}  // namespace slide_attn
