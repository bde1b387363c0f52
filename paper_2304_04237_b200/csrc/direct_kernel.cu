// DIRECT variant: one warp per (query pixel, head); keys and values are read straight from
// global memory with bounds checks (a position outside the map reads as zero, Fig. 2), all
// arithmetic in fp32 on the CUDA cores.  It accepts every supported shape and serves as the
// on-device cross-check of the faster variants.
//
// Per (pixel, head), with lane = channel within the head (strided by 32 when head_dim > 32):
//   logits l[s] = (1/sqrt(d)) * sum_c q[c] * sum_t wk[c,s,t] * K0(p+off(t), c) + bias[h,s]
//   a = softmax_s(l);  out[c] = sum_s a[s] * sum_t wv[c,s,t] * V0(p+off(t), c)      (Eq. 2, Eq. 12)
#include "common.cuh"

namespace slide_attn {

namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <typename T, int KS>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
direct_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
              const float* __restrict__ wk, const float* __restrict__ wv,
              const float* __restrict__ bias, T* __restrict__ out,
              int B, int H, int W, int heads, int d, float scale)
{
    constexpr int K2 = KS * KS;
    constexpr int R = KS / 2;
    __shared__ float s_logit[kWarpsPerBlock][K2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long units = (long long)B * H * W * heads;
    const long long unit = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (unit >= units) return;                       // whole warp leaves together

    const int h = (int)(unit % heads);
    const long long pix = unit / heads;
    const int j = (int)(pix % W);
    const int i = (int)((pix / W) % H);
    const int b = (int)(pix / ((long long)W * H));
    const int C = heads * d;
    const size_t px_base = (size_t)pix * C;
    float* logit = s_logit[warp];

    for (int s = lane; s < K2; s += 32) logit[s] = bias ? bias[h * K2 + s] : 0.f;
    __syncwarp();

    // ---- logits -------------------------------------------------------------------------
    for (int e0 = 0; e0 < d; e0 += 32) {
        const int e = e0 + lane;
        const bool live = e < d;
        const int c = h * d + (live ? e : 0);
        float kt[K2];
#pragma unroll
        for (int p = 0; p < KS; ++p)
#pragma unroll
            for (int q_ = 0; q_ < KS; ++q_) {
                const int ii = i + p - R, jj = j + q_ - R;
                const bool in = live && ii >= 0 && ii < H && jj >= 0 && jj < W;
                kt[p * KS + q_] = in ? to_float(k[(((size_t)b * H + ii) * W + jj) * C + c]) : 0.f;
            }
        const float qv = live ? to_float(q[px_base + c]) * scale : 0.f;
        const float* wrow = wk + (size_t)c * K2 * K2;
        for (int s = 0; s < K2; ++s) {
            float acc = 0.f;
#pragma unroll
            for (int t = 0; t < K2; ++t) acc = fmaf(wrow[s * K2 + t], kt[t], acc);
            const float part = warp_sum(qv * acc);
            if (lane == 0) logit[s] += part;
        }
    }
    __syncwarp();

    // ---- softmax over the k*k slots (every lane evaluates it; the row is tiny) -----------
    float m = -INFINITY;
    for (int s = 0; s < K2; ++s) m = fmaxf(m, logit[s]);
    float z = 0.f;
    for (int s = 0; s < K2; ++s) z += __expf(logit[s] - m);
    const float inv_z = 1.f / z;
    __syncwarp();
    for (int s = lane; s < K2; s += 32) logit[s] = __expf(logit[s] - m) * inv_z;
    __syncwarp();

    // ---- aggregation ---------------------------------------------------------------------
    for (int e0 = 0; e0 < d; e0 += 32) {
        const int e = e0 + lane;
        if (e >= d) break;
        const int c = h * d + e;
        float vt[K2];
#pragma unroll
        for (int p = 0; p < KS; ++p)
#pragma unroll
            for (int q_ = 0; q_ < KS; ++q_) {
                const int ii = i + p - R, jj = j + q_ - R;
                const bool in = ii >= 0 && ii < H && jj >= 0 && jj < W;
                vt[p * KS + q_] = in ? to_float(v[(((size_t)b * H + ii) * W + jj) * C + c]) : 0.f;
            }
        const float* wrow = wv + (size_t)c * K2 * K2;
        float o = 0.f;
        for (int s = 0; s < K2; ++s) {
            float acc = 0.f;
#pragma unroll
            for (int t = 0; t < K2; ++t) acc = fmaf(wrow[s * K2 + t], vt[t], acc);
            o = fmaf(logit[s], acc, o);
        }
        out[px_base + c] = from_float<T>(o);
    }
}

template <typename T, int KS>
cudaError_t launch_ks(const Problem& p, cudaStream_t stream) {
    const long long units = (long long)p.B * p.H * p.W * p.heads;
    const long long blocks = (units + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    direct_kernel<T, KS><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(
        (const T*)p.q, (const T*)p.k, (const T*)p.v, p.wk, p.wv, p.bias, (T*)p.out,
        p.B, p.H, p.W, p.heads, p.head_dim, rsqrtf((float)p.head_dim));
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(const Problem& p, cudaStream_t stream) {
    switch (p.ksize) {
        case 1:  return launch_ks<T, 1>(p, stream);
        case 3:  return launch_ks<T, 3>(p, stream);
        case 5:  return launch_ks<T, 5>(p, stream);
        case 7:  return launch_ks<T, 7>(p, stream);
        case 9:  return launch_ks<T, 9>(p, stream);
        case 11: return launch_ks<T, 11>(p, stream);
        case 13: return launch_ks<T, 13>(p, stream);
        case 15: return launch_ks<T, 15>(p, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool direct_supports(int head_dim, int ksize) {
    return head_dim >= 1 && ksize >= 1 && ksize <= 15 && (ksize & 1);
}

cudaError_t launch_direct(const Problem& p, cudaStream_t stream) {
    return p.dtype == SLIDE_ATTN_BF16 ? launch_t<__nv_bfloat16>(p, stream) : launch_t<float>(p, stream);
}

}  // namespace slide_attn
