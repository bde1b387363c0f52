// TILE variant: the generic fused forward (any merged depthwise weights, Eq. 2 with Eq. 12 inside) for
// head_dim 32, k <= 9, fp32 or bf16 storage, staged like the fixed-shift kernel: the K and V tile + halo
// and the q tile come in by TMA into shared memory (zero fill = the padding), every access to them is a
// conflict-free 16-byte load, the output goes out in 16-byte stores, and all arithmetic is fp32 on the
// CUDA cores (packed FMAs).  It is what AUTO runs where the tensor-core kernel does not apply (fp32
// storage, k >= 5).
//
// Per lane (column g, the eight channels of piece tig) and sub-strip of RS pixel rows, the convolution
// is never formed per slot; it is re-associated with the q.k product and with the attention weights:
//   logits   l[r][s] = sum_t sum_c (q[r][c] k[r + off(t)][c]) wk[c][s][t]
//            for every tap t: P[r][c] = q k (8 products), then for every slot s one 32-byte weight
//            vector feeds RS x 8 multiply-adds; partial sums over the lane's channels are completed
//            across the quad by shuffles
//   values   out[r][c] = sum_t v[r + off(t)][c] * (sum_s a[r][s] wv[c][s][t])
// Weights are read from the transposed copy [slot][tap][C] that the prep launch of every forward
// writes to the context workspace (all eight lanes of a column group read the same 128 bytes, which
// the L1 cache serves).  2 k^4 + 2 k^2 multiply-adds per pixel-channel: bound by the fp32 pipes.
#include "tile_common.cuh"

namespace slide_attn {

namespace {

using namespace tile;

// sub-strip height: the logits of RS pixels x k^2 slots live in registers as channel-parity pairs
template <int K> struct Strip { static constexpr int rs = K <= 3 ? 4 : (K <= 5 ? 2 : 1); };
// For k <= 3 the head's transposed weights (2 x k^4 x 32 floats = 20.7 KB) are copied to shared memory
// once per CTA; wider windows read them through the L1 cache.
template <int K> struct WeightHome { static constexpr bool smem = K <= 3; static constexpr uint32_t bytes = smem ? 2u * K * K * K * K * 128u : 0u; };

template <typename T> struct WeightVec;
template <> struct WeightVec<__nv_bfloat16> {       // channels 8 tig .. 8 tig + 7
    static __device__ __forceinline__ void load(const float* w, int tig, float (&f)[8]) {
        const float4 a = *reinterpret_cast<const float4*>(w + 8 * tig);
        const float4 b = *reinterpret_cast<const float4*>(w + 8 * tig + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
};
template <> struct WeightVec<float> {               // channels 4 tig .. 4 tig + 3 and 16 + 4 tig ..
    static __device__ __forceinline__ void load(const float* w, int tig, float (&f)[8]) {
        const float4 a = *reinterpret_cast<const float4*>(w + 4 * tig);
        const float4 b = *reinterpret_cast<const float4*>(w + 16 + 4 * tig);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
};

template <typename T, int K>
__global__ void __launch_bounds__(Cfg<T, K>::threads)
tile_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
            const __grid_constant__ CUtensorMap map_v, const TileParams P)
{
    using C_ = Cfg<T, K>;
    constexpr int R = K / 2, K2 = K * K, RS = Strip<K>::rs;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t bar = smem_u32(smem + C_::bar_off);
    float* s_bias = reinterpret_cast<float*>(smem + C_::bias_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int h = blockIdx.x % P.heads;
    int tile = blockIdx.x / P.heads;
    const int tx = tile % P.tiles_x; tile /= P.tiles_x;
    const int ty = tile % P.tiles_y;
    const int b = tile / P.tiles_y;
    const int x0 = tx * kTW, y0 = ty * C_::TH;
    constexpr int chan_per_plane = 64 / (int)sizeof(T);
    const int Ctot = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_expect_tx(bar, C_::tx_bytes);
#pragma unroll
        for (int pl = 0; pl < C_::planes; ++pl) {
            const int c0 = h * kHeadDim + pl * chan_per_plane;
            tma_load_4d(smem_u32(smem + C_::k_off + pl * C_::halo_plane), &map_k, bar, c0, x0 - R, y0 - R, b);
            tma_load_4d(smem_u32(smem + C_::v_off + pl * C_::halo_plane), &map_v, bar, c0, x0 - R, y0 - R, b);
            tma_load_4d(smem_u32(smem + C_::q_off + pl * C_::q_plane), &map_q, bar, c0, x0, y0, b);
        }
    }
    for (int i = threadIdx.x; i < K2; i += C_::threads) s_bias[i] = P.bias ? P.bias[h * K2 + i] * kLog2e : 0.f;
    if constexpr (WeightHome<K>::smem) {
        float4* dst = reinterpret_cast<float4*>(smem + C_::bar_off + 16);   // behind the barrier; the tail slack covers the alignment shift
        for (int i = threadIdx.x; i < 2 * K2 * K2 * 8; i += C_::threads) {
            const int st = i >> 3, part = i & 7;                 // (side, slot, tap) and 16-byte part of the 128 bytes
            dst[i] = __ldg(reinterpret_cast<const float4*>(P.wt + (size_t)st * Ctot + h * kHeadDim) + part);
        }
    }
    __syncthreads();
    if (!mbar_wait(bar, 0)) {                                  // bounded: about two seconds
        if (lane == 0) atomicExch(P.status, 1);
        return;
    }

    const int wx = warp % (kTW / 8), wy = warp / (kTW / 8);
    const int col = wx * 8 + g, row0 = wy * kR;
    const unsigned char* sK = smem + C_::k_off;
    const unsigned char* sV = smem + C_::v_off;
    const unsigned char* sQ = smem + C_::q_off;
    // weight vector of (slot s, tap t): wkt + (s K2 + t) wstride, 32 floats of this head
    const float* wkt;
    const float* wvt;
    int wstride;
    if constexpr (WeightHome<K>::smem) {
        wkt = reinterpret_cast<const float*>(smem + C_::bar_off + 16);
        wvt = wkt + K2 * K2 * kHeadDim;
        wstride = kHeadDim;
    } else {
        wkt = P.wt + h * kHeadDim;
        wvt = wkt + (size_t)Ctot * K2 * K2;
        wstride = Ctot;
    }
    const int x = x0 + col;

#pragma unroll 1
    for (int rs0 = 0; rs0 < kR; rs0 += RS) {
        float qf[RS][8];
#pragma unroll
        for (int r = 0; r < RS; ++r)
            Piece<T>::widen(Piece<T>::load(sQ, C_::q_plane, (uint32_t)((row0 + rs0 + r) * kTW + col), tig), qf[r]);

        // ---- logits: channel-parity pairs of partial sums over this lane's channels ----------------
        float l[RS][K2][2];
#pragma unroll
        for (int r = 0; r < RS; ++r)
#pragma unroll
            for (int s = 0; s < K2; ++s) { l[r][s][0] = 0.f; l[r][s][1] = 0.f; }
#pragma unroll 1
        for (int t = 0; t < K2; ++t) {
            const int ty_ = t / K, tx_ = t - ty_ * K;
            float pr[RS][8];
#pragma unroll
            for (int r = 0; r < RS; ++r) {
                float kv[8];
                Piece<T>::widen(Piece<T>::load(sK, C_::halo_plane, (uint32_t)((row0 + rs0 + r + ty_) * C_::HW + col + tx_), tig), kv);
#pragma unroll
                for (int c = 0; c < 8; ++c) pr[r][c] = qf[r][c] * kv[c];
            }
            const float* wp = wkt + (size_t)t * wstride;
#pragma unroll
            for (int s = 0; s < K2; ++s) {
                float w[8];
                WeightVec<T>::load(wp + (size_t)s * K2 * wstride, tig, w);
#pragma unroll
                for (int r = 0; r < RS; ++r)
#pragma unroll
                    for (int c = 0; c < 8; c += 2) ffma2(l[r][s][0], l[r][s][1], pr[r][c], pr[r][c + 1], w[c], w[c + 1]);
            }
        }
        // ---- complete the sums across the quad, softmax per pixel (every lane of the quad) ---------
        float a[RS][K2], inv[RS];
#pragma unroll
        for (int r = 0; r < RS; ++r) {
            float m = -INFINITY;
#pragma unroll
            for (int s = 0; s < K2; ++s) {
                float v = l[r][s][0] + l[r][s][1];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v = fmaf(v, P.scale_log2e, s_bias[s]);
                a[r][s] = v;
                m = fmaxf(m, v);
            }
            float z = 0.f;
#pragma unroll
            for (int s = 0; s < K2; ++s) { a[r][s] = fast_exp2(a[r][s] - m); z += a[r][s]; }
            inv[r] = 1.f / z;
        }
        // ---- values -------------------------------------------------------------------------------
        float acc[RS][8];
#pragma unroll
        for (int r = 0; r < RS; ++r)
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;
#pragma unroll 1
        for (int t = 0; t < K2; ++t) {
            const int ty_ = t / K, tx_ = t - ty_ * K;
            float aw[RS][8];                                     // sum_s a[r][s] wv[c][s][t]
#pragma unroll
            for (int r = 0; r < RS; ++r)
#pragma unroll
                for (int c = 0; c < 8; ++c) aw[r][c] = 0.f;
            const float* wp = wvt + (size_t)t * wstride;
#pragma unroll
            for (int s = 0; s < K2; ++s) {
                float w[8];
                WeightVec<T>::load(wp + (size_t)s * K2 * wstride, tig, w);
#pragma unroll
                for (int r = 0; r < RS; ++r) {
                    const float e = a[r][s];
#pragma unroll
                    for (int c = 0; c < 8; c += 2) ffma2(aw[r][c], aw[r][c + 1], e, e, w[c], w[c + 1]);
                }
            }
#pragma unroll
            for (int r = 0; r < RS; ++r) {
                float vv[8];
                Piece<T>::widen(Piece<T>::load(sV, C_::halo_plane, (uint32_t)((row0 + rs0 + r + ty_) * C_::HW + col + tx_), tig), vv);
#pragma unroll
                for (int c = 0; c < 8; c += 2) ffma2(acc[r][c], acc[r][c + 1], aw[r][c], aw[r][c + 1], vv[c], vv[c + 1]);
            }
        }
#pragma unroll
        for (int r = 0; r < RS; ++r) {
            const int y = y0 + row0 + rs0 + r;
            if (x < P.W && y < P.H) {
                const float iv = inv[r];
                const size_t base = ((size_t)(b * P.H + y) * P.W + x) * Ctot + h * kHeadDim;
                if constexpr (sizeof(T) == 2) {
                    uint4 o;
                    o.x = pack_bf16(acc[r][0] * iv, acc[r][1] * iv); o.y = pack_bf16(acc[r][2] * iv, acc[r][3] * iv);
                    o.z = pack_bf16(acc[r][4] * iv, acc[r][5] * iv); o.w = pack_bf16(acc[r][6] * iv, acc[r][7] * iv);
                    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + base + tig * 8) = o;
                } else {
                    float* op = static_cast<float*>(P.out) + base;
                    *reinterpret_cast<float4*>(op + tig * 4) = make_float4(acc[r][0] * iv, acc[r][1] * iv, acc[r][2] * iv, acc[r][3] * iv);
                    *reinterpret_cast<float4*>(op + 16 + tig * 4) = make_float4(acc[r][4] * iv, acc[r][5] * iv, acc[r][6] * iv, acc[r][7] * iv);
                }
            }
        }
    }
}

template <typename T, int K>
cudaError_t launch_t(const Problem& p, const float* wt, int* d_status, cudaStream_t stream) {
    using C_ = Cfg<T, K>;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(tile_kernel<T, K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(C_::total + WeightHome<K>::bytes));
        if (e != cudaSuccess) return e;
        if (dev < 64) configured[dev] = true;
    }
    TileParams P;
    P.wt = wt; P.bias = p.bias; P.out = p.out; P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.tiles_x = (p.W + kTW - 1) / kTW;
    P.tiles_y = (p.H + C_::TH - 1) / C_::TH;
    P.scale_log2e = kLog2e / sqrtf((float)kHeadDim);
    const int Ctot = p.heads * kHeadDim;
    const int cpp = 64 / (int)sizeof(T);
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, p.q, (int)sizeof(T), p.B, p.H, p.W, Ctot, cpp, kTW, C_::TH) ||
        !make_tile_map(&mk, p.k, (int)sizeof(T), p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH) ||
        !make_tile_map(&mv, p.v, (int)sizeof(T), p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH))
        return cudaErrorInvalidValue;
    const long long ctas = (long long)P.tiles_x * P.tiles_y * p.B * p.heads;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    tile_kernel<T, K><<<(unsigned)ctas, C_::threads, C_::total + WeightHome<K>::bytes, stream>>>(mq, mk, mv, P);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_k(const Problem& p, const float* wt, int* d_status, cudaStream_t stream) {
    switch (p.ksize) {
        case 1: return launch_t<T, 1>(p, wt, d_status, stream);
        case 3: return launch_t<T, 3>(p, wt, d_status, stream);
        case 5: return launch_t<T, 5>(p, wt, d_status, stream);
        case 7: return launch_t<T, 7>(p, wt, d_status, stream);
        case 9: return launch_t<T, 9>(p, wt, d_status, stream);
        default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace

bool tile_supports(int head_dim, int ksize) {
    return head_dim == kHeadDim && (ksize & 1) && ksize >= 1 && ksize <= 9 && tensor_map_available();
}

// `workspace`: the transposed weights written by launch_strip_prep (wk^T then wv^T, [slot][tap][C]).
cudaError_t launch_tile(const Problem& p, const void* workspace, int* d_status, cudaStream_t stream) {
    const float* wt = static_cast<const float*>(workspace);
    return p.dtype == SLIDE_ATTN_BF16 ? launch_k<__nv_bfloat16>(p, wt, d_status, stream) : launch_k<float>(p, wt, d_status, stream);
}

}  // namespace slide_attn
