// STRIP variant: the generic fp32 path for every shape the tensor-core variants do not take (other
// window sizes, other head widths, fp32 storage).  Same arithmetic as DIRECT (Eq. 2 with Eq. 12
// inside, no re-association), organised so that the CUDA cores are fed from registers and
// coalesced loads:
//   * a prep kernel transposes both weight tensors from [C][slot][tap] to [slot][tap][C], so that a
//     warp whose lanes are 32 consecutive channels reads one weight of each with ONE 128-byte load;
//   * one warp takes one head of a strip of eight (four for k >= 7) horizontally adjacent pixels: every
//     weight it loads is used for all of them, and the k x (k + strip - 1) window of keys (values) of a
//     lane's channel lives in registers for the whole strip.
// Per (pixel, head), lane = channel within the head (strided by 32 when head_dim > 32):
//   logits l[s] = (1/sqrt(d)) * sum_c q[c] * sum_t wk[c,s,t] * K0(p+off(t), c) + bias[h,s]
//   a = softmax_s(l);  out[c] = sum_s a[s] * sum_t wv[c,s,t] * V0(p+off(t), c)
// with K0 / V0 reading zero outside the map (Fig. 2).
#include "common.cuh"

namespace slide_attn {

namespace {

constexpr int kWarpsPerBlock = 4;

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// [C][K2][K2] -> [K2][K2][C] for both tensors; `dst` holds wk^T then wv^T.
__global__ void strip_prep_kernel(const float* __restrict__ wk, const float* __restrict__ wv,
                                  float* __restrict__ dst, int C, int K2)
{
    const long long n = (long long)C * K2 * K2;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < 2 * n;
         i += (long long)gridDim.x * blockDim.x) {
        const long long j = i < n ? i : i - n;                 // index into the transposed tensor
        const int c = (int)(j % C);
        const long long st = j / C;                            // slot * K2 + tap
        const float* src = i < n ? wk : wv;
        dst[i] = src[(long long)c * K2 * K2 + st];
    }
}

// kStrip = pixels per warp: 8 while the window fits the register file, 4 for the widest windows.
template <typename T, int KS, int kStrip>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
strip_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
             const float* __restrict__ wt,                   // transposed weights: wk^T, then wv^T
             const float* __restrict__ bias, T* __restrict__ out,
             int B, int H, int W, int heads, int d, float scale)
{
    constexpr int K2 = KS * KS;
    constexpr int R = KS / 2;
    constexpr int WC = KS + kStrip - 1;                       // window columns
    __shared__ float s_logit[kWarpsPerBlock][kStrip][K2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int strips_x = (W + kStrip - 1) / kStrip;
    const long long units = (long long)B * H * strips_x * heads;
    const long long unit = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (unit >= units) return;                                // whole warp leaves together

    const int h = (int)(unit % heads);
    long long rest = unit / heads;
    const int j0 = (int)(rest % strips_x) * kStrip;           // first column of the strip
    rest /= strips_x;
    const int i = (int)(rest % H);
    const int b = (int)(rest / H);
    const int C = heads * d;
    const size_t row_base = ((size_t)b * H + i) * W;          // pixel index of (b, i, 0)
    const float* wkt = wt;
    const float* wvt = wt + (size_t)C * K2 * K2;
    float (*logit)[K2] = s_logit[warp];

    for (int x = lane; x < kStrip * K2; x += 32) logit[x / K2][x % K2] = bias ? bias[h * K2 + x % K2] : 0.f;
    __syncwarp();

    // the k x (k + strip - 1) window of one channel around the strip, zero outside the map
    auto load_window = [&](const T* __restrict__ src, int c, bool live, float (&win)[KS][WC]) {
#pragma unroll
        for (int r = 0; r < KS; ++r) {
            const int ii = i + r - R;
#pragma unroll
            for (int cc = 0; cc < WC; ++cc) {
                const int jj = j0 + cc - R;
                const bool in = live && ii >= 0 && ii < H && jj >= 0 && jj < W;
                win[r][cc] = in ? to_float(src[(((size_t)b * H + ii) * W + jj) * C + c]) : 0.f;
            }
        }
    };

    // ---- logits -------------------------------------------------------------------------
    for (int e0 = 0; e0 < d; e0 += 32) {
        const int e = e0 + lane;
        const bool live = e < d;
        const int c = h * d + (live ? e : 0);
        float win[KS][WC];
        load_window(k, c, live, win);
        float qv[kStrip];
#pragma unroll
        for (int p = 0; p < kStrip; ++p)
            qv[p] = (live && j0 + p < W) ? to_float(q[(row_base + j0 + p) * C + c]) * scale : 0.f;
        const float* wc = wkt + c;
        for (int s = 0; s < K2; ++s) {
            float acc[kStrip];
#pragma unroll
            for (int p = 0; p < kStrip; ++p) acc[p] = 0.f;
#pragma unroll
            for (int r = 0; r < KS; ++r)
#pragma unroll
                for (int cc = 0; cc < KS; ++cc) {
                    const float w = wc[(size_t)(s * K2 + r * KS + cc) * C];
#pragma unroll
                    for (int p = 0; p < kStrip; ++p) acc[p] = fmaf(w, win[r][cc + p], acc[p]);
                }
#pragma unroll
            for (int p = 0; p < kStrip; ++p) {
                const float part = warp_sum(qv[p] * acc[p]);
                if (lane == 0) logit[p][s] += part;
            }
        }
    }
    __syncwarp();

    // ---- softmax over the k*k slots of each pixel (every lane evaluates it; the rows are tiny) ---
#pragma unroll
    for (int p = 0; p < kStrip; ++p) {
        float m = -INFINITY;
        for (int s = 0; s < K2; ++s) m = fmaxf(m, logit[p][s]);
        float z = 0.f;
        for (int s = 0; s < K2; ++s) z += __expf(logit[p][s] - m);
        const float inv_z = 1.f / z;
        __syncwarp();
        for (int s = lane; s < K2; s += 32) logit[p][s] = __expf(logit[p][s] - m) * inv_z;
    }
    __syncwarp();

    // ---- aggregation ---------------------------------------------------------------------
    for (int e0 = 0; e0 < d; e0 += 32) {
        const int e = e0 + lane;
        if (e >= d) break;
        const int c = h * d + e;
        float win[KS][WC];
        load_window(v, c, true, win);
        const float* wc = wvt + c;
        float o[kStrip];
#pragma unroll
        for (int p = 0; p < kStrip; ++p) o[p] = 0.f;
        for (int s = 0; s < K2; ++s) {
            float acc[kStrip];
#pragma unroll
            for (int p = 0; p < kStrip; ++p) acc[p] = 0.f;
#pragma unroll
            for (int r = 0; r < KS; ++r)
#pragma unroll
                for (int cc = 0; cc < KS; ++cc) {
                    const float w = wc[(size_t)(s * K2 + r * KS + cc) * C];
#pragma unroll
                    for (int p = 0; p < kStrip; ++p) acc[p] = fmaf(w, win[r][cc + p], acc[p]);
                }
#pragma unroll
            for (int p = 0; p < kStrip; ++p) o[p] = fmaf(logit[p][s], acc[p], o[p]);
        }
#pragma unroll
        for (int p = 0; p < kStrip; ++p)
            if (j0 + p < W) out[(row_base + j0 + p) * C + c] = from_float<T>(o[p]);
    }
}

template <typename T, int KS>
cudaError_t launch_ks(const Problem& p, const float* wt, cudaStream_t stream) {
    constexpr int kStrip = KS <= 5 ? 8 : 4;
    const long long units = (long long)p.B * p.H * ((p.W + kStrip - 1) / kStrip) * p.heads;
    const long long blocks = (units + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    strip_kernel<T, KS, kStrip><<<(unsigned)blocks, kWarpsPerBlock * 32, 0, stream>>>(
        (const T*)p.q, (const T*)p.k, (const T*)p.v, wt, p.bias, (T*)p.out,
        p.B, p.H, p.W, p.heads, p.head_dim, rsqrtf((float)p.head_dim));
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(const Problem& p, const float* wt, cudaStream_t stream) {
    switch (p.ksize) {
        case 1: return launch_ks<T, 1>(p, wt, stream);
        case 3: return launch_ks<T, 3>(p, wt, stream);
        case 5: return launch_ks<T, 5>(p, wt, stream);
        case 7: return launch_ks<T, 7>(p, wt, stream);
        case 9: return launch_ks<T, 9>(p, wt, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool strip_supports(int head_dim, int ksize) {
    return head_dim >= 1 && (ksize & 1) && ksize >= 1 && ksize <= 9;   // wider windows: DIRECT
}

size_t strip_workspace_bytes(int heads, int head_dim, int ksize) {
    const size_t k2 = (size_t)ksize * ksize;
    return 2 * (size_t)heads * head_dim * k2 * k2 * sizeof(float);
}

cudaError_t launch_strip_prep(const Problem& p, void* workspace, cudaStream_t stream) {
    const int C = p.heads * p.head_dim, K2 = p.ksize * p.ksize;
    const long long n = 2LL * C * K2 * K2;
    const int threads = 256;
    long long blocks = (n + threads - 1) / threads;
    if (blocks > 4096) blocks = 4096;
    strip_prep_kernel<<<(unsigned)blocks, threads, 0, stream>>>(p.wk, p.wv, static_cast<float*>(workspace), C, K2);
    return cudaGetLastError();
}

cudaError_t launch_strip_main(const Problem& p, const void* workspace, cudaStream_t stream) {
    const float* wt = static_cast<const float*>(workspace);
    return p.dtype == SLIDE_ATTN_BF16 ? launch_t<__nv_bfloat16>(p, wt, stream) : launch_t<float>(p, wt, stream);
}

}  // namespace slide_attn
