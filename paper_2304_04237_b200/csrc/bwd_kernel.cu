// Backward pass of the fused forward (training through the module, Sec. 4.3 / Fig. 4 (1); the paper
// prints no backward formulas: these are the derivatives of Eq. 2 with the depthwise convolution of
// Eq. 12 inside).  head_dim 32, k = 1 or 3, fp32 or bf16 storage, fp32 arithmetic on the CUDA cores,
// staged like tile_kernel (TMA halo tiles in 64-byte channel planes, lane = column g x the eight
// channels of piece tig, a warp = 8 columns x 4 rows).  With g = d(loss)/d(out):
//
//   forward again   a = softmax_s( scale * sum_{t,c} q[c] k_t[c] wk[c,s,t] + bias[s] )
//   da[s]   = sum_{t,c} g[c] v_t[c] wv[c,s,t]                 (the logit contraction with g, v, wv)
//   dl[s]   = a[s] (da[s] - sum_s' a[s'] da[s'])
//   dbias[s] = sum over pixels of dl[s]
//   dq[c]   = scale * sum_t k_t[c] (sum_s dl[s] wk[c,s,t])     (the value contraction with dl, wk, k)
//   dwk[c,s,t] = scale * sum over pixels of dl[s] q[c] k_t[c]      dwv[c,s,t] = sum a[s] g[c] v_t[c]
//   dk[p'][c] = scale * sum_t q[p' - off(t)][c] (sum_s dl[p' - off(t)][s] wk[c,s,t])     (gather form of the
//   dv[p'][c] =         sum_t g[p' - off(t)][c] (sum_s  a[p' - off(t)][s] wv[c,s,t])      transposed shift)
//
// Three kernels.  bwd_point_kernel does what belongs to the query pixel: a, dl (kept in a workspace for
// the other two), dq and the bias gradient.  bwd_gather_kernel computes dk and dv per key / value pixel by
// gathering from the k x k query pixels whose windows hold it (out-of-map queries contribute nothing:
// their q, g tiles read as zero).  bwd_weight_kernel (persistent CTAs, one head each) sums the weight
// gradients over the pixels with lane = channel, so that a lane's 2 k^4 accumulators live in registers
// over all its tiles and no reduction across lanes is needed; one addition per weight and CTA goes to
// global memory at its end.
#include "tile_common.cuh"

namespace slide_attn {

namespace {

using namespace tile;

struct BwdParams {
    const float* wt;                 // transposed weights wk^T then wv^T, [slot][tap][C]
    const float* bias;
    void* dq;
    void* dk;
    void* dv;
    float* dwk;
    float* dwv;
    float* dbias;
    float* ws_a;                     // [pixel][head][k*k]
    float* ws_dl;
    int* status;
    int B, H, W, heads;
    int tiles_x, tiles_y;
    float scale;                     // 1 / sqrt(head_dim)
};

// the lane's eight weights of one (slot, tap) vector of 32 floats, and the same addressing for adds
template <typename T> struct WVec;
template <> struct WVec<__nv_bfloat16> {
    static __device__ __forceinline__ int chan(int tig, int c) { return 8 * tig + c; }
};
template <> struct WVec<float> {
    static __device__ __forceinline__ int chan(int tig, int c) { return c < 4 ? 4 * tig + c : 16 + 4 * tig + (c - 4); }
};
template <typename T>
__device__ __forceinline__ void wload(const float* w, int tig, float (&f)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(w + WVec<T>::chan(tig, 0));
    const float4 b = *reinterpret_cast<const float4*>(w + WVec<T>::chan(tig, 4));
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

template <typename T>
__device__ __forceinline__ void store8(void* base, size_t elem, int tig, const float (&f)[8]) {
    if constexpr (sizeof(T) == 2) {
        uint4 o;
        o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]); o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + elem + tig * 8) = o;
    } else {
        float* op = static_cast<float*>(base) + elem;
        *reinterpret_cast<float4*>(op + tig * 4) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4*>(op + 16 + tig * 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
}

template <typename T, int K>
struct PointCfg {
    using C_ = Cfg<T, K>;
    static constexpr int K2 = K * K;
    static constexpr uint32_t k_off = 0, v_off = C_::planes * C_::halo_plane;
    static constexpr uint32_t q_off = 2 * C_::planes * C_::halo_plane, g_off = q_off + C_::planes * C_::q_plane;
    static constexpr uint32_t w_off = g_off + C_::planes * C_::q_plane;              // weights [2][K2*K2][32] floats
    static constexpr uint32_t bias_off = w_off + 2u * K2 * K2 * 128u;                // bias (log2 units), then dbias
    static constexpr uint32_t bar_off = bias_off + ((2 * K2 * 4 + 15) & ~15);
    static constexpr uint32_t total = bar_off + 16 + 128;
    static constexpr uint32_t tx_bytes = C_::planes * (2u * C_::HW * C_::HH * 64u + 2u * C_::q_plane);
};

template <typename T, int K>
__global__ void __launch_bounds__(Cfg<T, K>::threads)
bwd_point_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_g,
                 const BwdParams P)
{
    using C_ = Cfg<T, K>;
    using L = PointCfg<T, K>;
    constexpr int R = K / 2, K2 = K * K;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t bar = smem_u32(smem + L::bar_off);
    float* s_w = reinterpret_cast<float*>(smem + L::w_off);
    float* s_bias = reinterpret_cast<float*>(smem + L::bias_off);
    float* s_dbias = s_bias + K2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int h = blockIdx.x % P.heads;
    int rest = blockIdx.x / P.heads;
    const int tx = rest % P.tiles_x; rest /= P.tiles_x;
    const int ty = rest % P.tiles_y;
    const int b = rest / P.tiles_y;
    const int x0 = tx * kTW, y0 = ty * C_::TH;
    constexpr int chan_per_plane = 64 / (int)sizeof(T);
    const int Ctot = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_expect_tx(bar, L::tx_bytes);
#pragma unroll
        for (int pl = 0; pl < C_::planes; ++pl) {
            const int c0 = h * kHeadDim + pl * chan_per_plane;
            tma_load_4d(smem_u32(smem + L::k_off + pl * C_::halo_plane), &map_k, bar, c0, x0 - R, y0 - R, b);
            tma_load_4d(smem_u32(smem + L::v_off + pl * C_::halo_plane), &map_v, bar, c0, x0 - R, y0 - R, b);
            tma_load_4d(smem_u32(smem + L::q_off + pl * C_::q_plane), &map_q, bar, c0, x0, y0, b);
            tma_load_4d(smem_u32(smem + L::g_off + pl * C_::q_plane), &map_g, bar, c0, x0, y0, b);
        }
    }
    for (int i = threadIdx.x; i < K2; i += C_::threads) { s_bias[i] = P.bias ? P.bias[h * K2 + i] * kLog2e : 0.f; s_dbias[i] = 0.f; }
    for (int i = threadIdx.x; i < 2 * K2 * K2 * 8; i += C_::threads) {
        const int st = i >> 3, part = i & 7;
        reinterpret_cast<float4*>(s_w)[i] = __ldg(reinterpret_cast<const float4*>(P.wt + (size_t)st * Ctot + h * kHeadDim) + part);
    }
    __syncthreads();
    if (!mbar_wait(bar, 0)) {                                    // bounded
        if (lane == 0) atomicExch(P.status, 1);
        return;
    }

    const int wx = warp % (kTW / 8), wy = warp / (kTW / 8);
    const int col = wx * 8 + g, row0 = wy * kR;
    const unsigned char* sK = smem + L::k_off;
    const unsigned char* sV = smem + L::v_off;
    const unsigned char* sQ = smem + L::q_off;
    const unsigned char* sG = smem + L::g_off;
    const float* wk_s = s_w;                                   // + (s K2 + t) 32
    const float* wv_s = s_w + K2 * K2 * kHeadDim;
    const float scale_log2e = P.scale * kLog2e;
    {
        float qf[kR][8], gf[kR][8];
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            Piece<T>::widen(Piece<T>::load(sQ, C_::q_plane, (uint32_t)((row0 + r) * kTW + col), tig), qf[r]);
            Piece<T>::widen(Piece<T>::load(sG, C_::q_plane, (uint32_t)((row0 + r) * kTW + col), tig), gf[r]);
        }
        // out[r][s] = sum_t sum_c A[r][c] B[r + off(t)][c] w[c][s][t], completed across the quad
        auto contract = [&](const float (&A)[kR][8], const unsigned char* halo, const float* wside, float (&out)[kR][K2]) {
            float l[kR][K2][2];
#pragma unroll
            for (int r = 0; r < kR; ++r)
#pragma unroll
                for (int s = 0; s < K2; ++s) { l[r][s][0] = 0.f; l[r][s][1] = 0.f; }
#pragma unroll 1
            for (int t = 0; t < K2; ++t) {
                const int ty_ = t / K, tx_ = t - ty_ * K;
                float pr[kR][8];
#pragma unroll
                for (int r = 0; r < kR; ++r) {
                    float kv[8];
                    Piece<T>::widen(Piece<T>::load(halo, C_::halo_plane, (uint32_t)((row0 + r + ty_) * C_::HW + col + tx_), tig), kv);
#pragma unroll
                    for (int c = 0; c < 8; ++c) pr[r][c] = A[r][c] * kv[c];
                }
#pragma unroll
                for (int s = 0; s < K2; ++s) {
                    float w[8];
                    wload<T>(wside + (s * K2 + t) * kHeadDim, tig, w);
#pragma unroll
                    for (int r = 0; r < kR; ++r)
#pragma unroll
                        for (int c = 0; c < 8; c += 2) ffma2(l[r][s][0], l[r][s][1], pr[r][c], pr[r][c + 1], w[c], w[c + 1]);
                }
            }
#pragma unroll
            for (int r = 0; r < kR; ++r)
#pragma unroll
                for (int s = 0; s < K2; ++s) {
                    float v = l[r][s][0] + l[r][s][1];
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    out[r][s] = v;
                }
        };

        float a[kR][K2], dl[kR][K2];
        contract(qf, sK, wk_s, a);
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            float m = -INFINITY, z = 0.f;
#pragma unroll
            for (int s = 0; s < K2; ++s) { a[r][s] = fmaf(a[r][s], scale_log2e, s_bias[s]); m = fmaxf(m, a[r][s]); }
#pragma unroll
            for (int s = 0; s < K2; ++s) { a[r][s] = fast_exp2(a[r][s] - m); z += a[r][s]; }
            const float iz = 1.f / z;
#pragma unroll
            for (int s = 0; s < K2; ++s) a[r][s] *= iz;
        }
        contract(gf, sV, wv_s, dl);                                  // da
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            float mean = 0.f;
#pragma unroll
            for (int s = 0; s < K2; ++s) mean = fmaf(a[r][s], dl[r][s], mean);
#pragma unroll
            for (int s = 0; s < K2; ++s) dl[r][s] = a[r][s] * (dl[r][s] - mean);
        }

        // ---- dq, and a / dl for the gather kernel -----------------------------------------------------
        {
            float acc[kR][8];
#pragma unroll
            for (int r = 0; r < kR; ++r)
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;
#pragma unroll 1
            for (int t = 0; t < K2; ++t) {
                const int ty_ = t / K, tx_ = t - ty_ * K;
                float aw[kR][8];
#pragma unroll
                for (int r = 0; r < kR; ++r)
#pragma unroll
                    for (int c = 0; c < 8; ++c) aw[r][c] = 0.f;
#pragma unroll
                for (int s = 0; s < K2; ++s) {
                    float w[8];
                    wload<T>(wk_s + (s * K2 + t) * kHeadDim, tig, w);
#pragma unroll
                    for (int r = 0; r < kR; ++r) {
                        const float e = dl[r][s];
#pragma unroll
                        for (int c = 0; c < 8; c += 2) ffma2(aw[r][c], aw[r][c + 1], e, e, w[c], w[c + 1]);
                    }
                }
#pragma unroll
                for (int r = 0; r < kR; ++r) {
                    float kv[8];
                    Piece<T>::widen(Piece<T>::load(sK, C_::halo_plane, (uint32_t)((row0 + r + ty_) * C_::HW + col + tx_), tig), kv);
#pragma unroll
                    for (int c = 0; c < 8; c += 2) ffma2(acc[r][c], acc[r][c + 1], aw[r][c], aw[r][c + 1], kv[c], kv[c + 1]);
                }
            }
            const int x = x0 + col;
#pragma unroll
            for (int r = 0; r < kR; ++r) {
                const int y = y0 + row0 + r;
                if (x < P.W && y < P.H) {
                    const size_t pix = (size_t)(b * P.H + y) * P.W + x;
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc[r][c] *= P.scale;
                    store8<T>(P.dq, pix * Ctot + h * kHeadDim, tig, acc[r]);
                    if (tig == 0) {
                        float* pa = P.ws_a + (pix * P.heads + h) * K2;
                        float* pd = P.ws_dl + (pix * P.heads + h) * K2;
#pragma unroll
                        for (int s = 0; s < K2; ++s) { pa[s] = a[r][s]; pd[s] = dl[r][s]; }
                    }
                }
            }
        }
        // ---- bias gradient: every lane of a quad holds the same dl; one lane per column counts ----------
        if (P.dbias) {
#pragma unroll
            for (int s = 0; s < K2; ++s) {
                float v = tig == 0 ? dl[0][s] + dl[1][s] + dl[2][s] + dl[3][s] : 0.f;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) atomicAdd(&s_dbias[s], v);
            }
        }
    }
    __syncthreads();
    if (P.dbias)
        for (int i = threadIdx.x; i < K2; i += C_::threads) atomicAdd(&P.dbias[h * K2 + i], s_dbias[i]);
}

// ---------------------------------------------------------------------------------------------------
// Weight gradients.  Persistent: CTA (head h, rank) walks tiles rank, rank + nrank, ...; warp w takes
// pixel row w of a tile, lane = channel.  Per pixel: P_t = q k_t and G_t = g v_t for the nine taps, then
// acc_k[s][t] += dl[s] P_t, acc_v[s][t] += a[s] G_t with dl, a broadcast from shared memory.
template <typename T, int K>
struct WeightCfg {
    using C_ = Cfg<T, K>;
    static constexpr int K2 = K * K;
    static constexpr uint32_t k_off = 0, v_off = C_::planes * C_::halo_plane;
    static constexpr uint32_t q_off = 2 * C_::planes * C_::halo_plane, g_off = q_off + C_::planes * C_::q_plane;
    static constexpr uint32_t a_off = g_off + C_::planes * C_::q_plane;                // [tile pixel][K2] a, then dl
    static constexpr uint32_t a_bytes = (uint32_t)(kTW * C_::TH * K2 * 4);
    static constexpr uint32_t dw_off = a_off + 2 * a_bytes;                           // [2][K2*K2][32] floats
    static constexpr uint32_t bar_off = dw_off + 2u * K2 * K2 * 128u;
    static constexpr uint32_t total = bar_off + 16 + 128;
    static constexpr uint32_t tx_bytes = C_::planes * (2u * C_::HW * C_::HH * 64u + 2u * C_::q_plane);
};

// element `c` (channel within the head) of pixel `pix` of a tile stored in 64-byte channel planes
template <typename T>
__device__ __forceinline__ float chan_load(const unsigned char* tile, uint32_t plane_bytes, uint32_t pix, int c) {
    if constexpr (sizeof(T) == 2)
        return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(tile + pix * 64u + c * 2u));
    else
        return *reinterpret_cast<const float*>(tile + (c >> 4) * plane_bytes + pix * 64u + (c & 15) * 4u);
}

template <typename T, int K>
__global__ void __launch_bounds__(Cfg<T, K>::threads)
bwd_weight_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_g,
                  const BwdParams P)
{
    using C_ = Cfg<T, K>;
    using L = WeightCfg<T, K>;
    constexpr int R = K / 2, K2 = K * K;
    static_assert(C_::TH == C_::warps, "one pixel row per warp");
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t bar = smem_u32(smem + L::bar_off);
    float* s_a = reinterpret_cast<float*>(smem + L::a_off);
    float* s_dl = reinterpret_cast<float*>(smem + L::a_off + L::a_bytes);
    float* s_dw = reinterpret_cast<float*>(smem + L::dw_off);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.x % P.heads;
    const int rank = blockIdx.x / P.heads;
    const int nrank = ((int)gridDim.x - h + P.heads - 1) / P.heads;
    const int tiles_per_head = P.B * P.tiles_y * P.tiles_x;
    constexpr int chan_per_plane = 64 / (int)sizeof(T);

    for (int i = threadIdx.x; i < 2 * K2 * K2 * kHeadDim; i += C_::threads) s_dw[i] = 0.f;
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();

    float acck[K2][K2], accv[K2][K2];                            // [slot][tap] of channel `lane`
#pragma unroll
    for (int s = 0; s < K2; ++s)
#pragma unroll
        for (int t = 0; t < K2; ++t) { acck[s][t] = 0.f; accv[s][t] = 0.f; }
    const unsigned char* sK = smem + L::k_off;
    const unsigned char* sV = smem + L::v_off;
    const unsigned char* sQ = smem + L::q_off;
    const unsigned char* sG = smem + L::g_off;
    bool ok = true;
    int it = 0;
    for (int tile = rank; tile < tiles_per_head; tile += nrank, ++it) {
        int rest = tile;
        const int tx = rest % P.tiles_x; rest /= P.tiles_x;
        const int ty = rest % P.tiles_y;
        const int b = rest / P.tiles_y;
        const int x0 = tx * kTW, y0 = ty * C_::TH;
        if (threadIdx.x == 0) {
            mbar_expect_tx(bar, L::tx_bytes);
#pragma unroll
            for (int pl = 0; pl < C_::planes; ++pl) {
                const int c0 = h * kHeadDim + pl * chan_per_plane;
                tma_load_4d(smem_u32(smem + L::k_off + pl * C_::halo_plane), &map_k, bar, c0, x0 - R, y0 - R, b);
                tma_load_4d(smem_u32(smem + L::v_off + pl * C_::halo_plane), &map_v, bar, c0, x0 - R, y0 - R, b);
                tma_load_4d(smem_u32(smem + L::q_off + pl * C_::q_plane), &map_q, bar, c0, x0, y0, b);
                tma_load_4d(smem_u32(smem + L::g_off + pl * C_::q_plane), &map_g, bar, c0, x0, y0, b);
            }
        }
        // a and dl of the tile's pixels (zero outside the map)
        for (int i = threadIdx.x; i < kTW * C_::TH; i += C_::threads) {
            const int py = i / kTW, px = i - py * kTW;
            const int y = y0 + py, x = x0 + px;
            const bool in = y < P.H && x < P.W;
            const size_t src = in ? (((size_t)(b * P.H + y) * P.W + x) * P.heads + h) * K2 : 0;
#pragma unroll
            for (int s = 0; s < K2; ++s) {
                s_a[i * K2 + s] = in ? P.ws_a[src + s] : 0.f;
                s_dl[i * K2 + s] = in ? P.ws_dl[src + s] : 0.f;
            }
        }
        __syncthreads();
        if (!mbar_wait(bar, (uint32_t)it & 1u)) { ok = false; break; }      // bounded

#pragma unroll 1
        for (int px = 0; px < kTW; ++px) {
            const uint32_t pix = (uint32_t)(warp * kTW + px);
            const float qv = chan_load<T>(sQ, C_::q_plane, pix, lane), gv = chan_load<T>(sG, C_::q_plane, pix, lane);
            float dls[K2], as[K2];
#pragma unroll
            for (int s = 0; s < K2; ++s) { dls[s] = s_dl[pix * K2 + s]; as[s] = s_a[pix * K2 + s]; }
#pragma unroll
            for (int t = 0; t < K2; ++t) {
                const uint32_t hp = (uint32_t)((warp + t / K) * C_::HW + px + t % K);
                const float pk = qv * chan_load<T>(sK, C_::halo_plane, hp, lane);
                const float pv = gv * chan_load<T>(sV, C_::halo_plane, hp, lane);
#pragma unroll
                for (int s = 0; s < K2; ++s) {
                    acck[s][t] = fmaf(dls[s], pk, acck[s][t]);
                    accv[s][t] = fmaf(as[s], pv, accv[s][t]);
                }
            }
        }
        __syncthreads();                                             // the tiles are free for the next load
    }
    if (!ok && lane == 0) atomicExch(P.status, 1);
    // the four warps' sums meet in shared memory, then one addition per weight into global memory
#pragma unroll
    for (int s = 0; s < K2; ++s)
#pragma unroll
        for (int t = 0; t < K2; ++t) {
            atomicAdd(&s_dw[(s * K2 + t) * kHeadDim + lane], acck[s][t]);
            atomicAdd(&s_dw[(K2 * K2 + s * K2 + t) * kHeadDim + lane], accv[s][t]);
        }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * K2 * K2 * kHeadDim; i += C_::threads) {
        const int side = i / (K2 * K2 * kHeadDim), rem = i - side * K2 * K2 * kHeadDim;
        const int st = rem / kHeadDim, ch = rem - st * kHeadDim;
        float* dst = (side == 0 ? P.dwk : P.dwv) + (size_t)(h * kHeadDim + ch) * K2 * K2 + st;
        atomicAdd(dst, side == 0 ? s_dw[i] * P.scale : s_dw[i]);
    }
}

template <typename T, int K>
struct GatherCfg {
    using C_ = Cfg<T, K>;
    static constexpr int K2 = K * K;
    static constexpr uint32_t q_off = 0, g_off = C_::planes * C_::halo_plane;        // both WITH halo
    static constexpr uint32_t w_off = 2 * C_::planes * C_::halo_plane;
    static constexpr uint32_t a_off = w_off + 2u * K2 * K2 * 128u;                    // [halo pixel][K2] a, then dl
    static constexpr uint32_t a_bytes = ((uint32_t)(C_::HW * C_::HH * K2 * 4) + 15u) & ~15u;
    static constexpr uint32_t bar_off = a_off + 2 * a_bytes;
    static constexpr uint32_t total = bar_off + 16 + 128;
    static constexpr uint32_t tx_bytes = C_::planes * 2u * C_::HW * C_::HH * 64u;
};

template <typename T, int K>
__global__ void __launch_bounds__(Cfg<T, K>::threads)
bwd_gather_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_g, const BwdParams P)
{
    using C_ = Cfg<T, K>;
    using L = GatherCfg<T, K>;
    constexpr int R = K / 2, K2 = K * K;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t bar = smem_u32(smem + L::bar_off);
    float* s_w = reinterpret_cast<float*>(smem + L::w_off);
    float* s_a = reinterpret_cast<float*>(smem + L::a_off);
    float* s_dl = reinterpret_cast<float*>(smem + L::a_off + L::a_bytes);

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
        mbar_expect_tx(bar, L::tx_bytes);
#pragma unroll
        for (int pl = 0; pl < C_::planes; ++pl) {
            const int c0 = h * kHeadDim + pl * chan_per_plane;
            tma_load_4d(smem_u32(smem + L::q_off + pl * C_::halo_plane), &map_q, bar, c0, x0 - R, y0 - R, b);
            tma_load_4d(smem_u32(smem + L::g_off + pl * C_::halo_plane), &map_g, bar, c0, x0 - R, y0 - R, b);
        }
    }
    for (int i = threadIdx.x; i < 2 * K2 * K2 * 8; i += C_::threads) {
        const int st = i >> 3, part = i & 7;
        reinterpret_cast<float4*>(s_w)[i] = __ldg(reinterpret_cast<const float4*>(P.wt + (size_t)st * Ctot + h * kHeadDim) + part);
    }
    // a and dl of the halo's query pixels; pixels outside the map hold zeros
    for (int i = threadIdx.x; i < C_::HW * C_::HH; i += C_::threads) {
        const int hy = i / C_::HW, hx = i - hy * C_::HW;
        const int y = y0 - R + hy, x = x0 - R + hx;
        const bool in = y >= 0 && y < P.H && x >= 0 && x < P.W;
        const size_t src = in ? (((size_t)(b * P.H + y) * P.W + x) * P.heads + h) * K2 : 0;
#pragma unroll
        for (int s = 0; s < K2; ++s) {
            s_a[i * K2 + s] = in ? P.ws_a[src + s] : 0.f;
            s_dl[i * K2 + s] = in ? P.ws_dl[src + s] : 0.f;
        }
    }
    __syncthreads();
    if (!mbar_wait(bar, 0)) {                                    // bounded
        if (lane == 0) atomicExch(P.status, 1);
        return;
    }

    const int wx = warp % (kTW / 8), wy = warp / (kTW / 8);
    const int col = wx * 8 + g, row0 = wy * kR;
    const unsigned char* sQ = smem + L::q_off;
    const unsigned char* sG = smem + L::g_off;
    const float* wk_s = s_w;
    const float* wv_s = s_w + K2 * K2 * kHeadDim;

    float dk[kR][8], dv[kR][8];
#pragma unroll
    for (int r = 0; r < kR; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) { dk[r][c] = 0.f; dv[r][c] = 0.f; }
#pragma unroll 1
    for (int t = 0; t < K2; ++t) {
        const int ty_ = t / K, tx_ = t - ty_ * K;
        // the query pixel whose tap t reads this key pixel: p = p' - off(t); halo coordinates (+R) of p
        const int hy0 = row0 + 2 * R - ty_, hx = col + 2 * R - tx_;
        float awk[kR][8], awv[kR][8];
#pragma unroll
        for (int r = 0; r < kR; ++r)
#pragma unroll
            for (int c = 0; c < 8; ++c) { awk[r][c] = 0.f; awv[r][c] = 0.f; }
#pragma unroll
        for (int s = 0; s < K2; ++s) {
            float w1[8], w2[8];
            wload<T>(wk_s + (s * K2 + t) * kHeadDim, tig, w1);
            wload<T>(wv_s + (s * K2 + t) * kHeadDim, tig, w2);
#pragma unroll
            for (int r = 0; r < kR; ++r) {
                const int hp = (hy0 + r) * C_::HW + hx;
                const float e1 = s_dl[hp * K2 + s], e2 = s_a[hp * K2 + s];
#pragma unroll
                for (int c = 0; c < 8; c += 2) {
                    ffma2(awk[r][c], awk[r][c + 1], e1, e1, w1[c], w1[c + 1]);
                    ffma2(awv[r][c], awv[r][c + 1], e2, e2, w2[c], w2[c + 1]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            const uint32_t hp = (uint32_t)((hy0 + r) * C_::HW + hx);
            float qv[8], gv[8];
            Piece<T>::widen(Piece<T>::load(sQ, C_::halo_plane, hp, tig), qv);
            Piece<T>::widen(Piece<T>::load(sG, C_::halo_plane, hp, tig), gv);
#pragma unroll
            for (int c = 0; c < 8; c += 2) {
                ffma2(dk[r][c], dk[r][c + 1], awk[r][c], awk[r][c + 1], qv[c], qv[c + 1]);
                ffma2(dv[r][c], dv[r][c + 1], awv[r][c], awv[r][c + 1], gv[c], gv[c + 1]);
            }
        }
    }
    const int x = x0 + col;
#pragma unroll
    for (int r = 0; r < kR; ++r) {
        const int y = y0 + row0 + r;
        if (x < P.W && y < P.H) {
            const size_t elem = ((size_t)(b * P.H + y) * P.W + x) * Ctot + h * kHeadDim;
#pragma unroll
            for (int c = 0; c < 8; ++c) dk[r][c] *= P.scale;
            store8<T>(P.dk, elem, tig, dk[r]);
            store8<T>(P.dv, elem, tig, dv[r]);
        }
    }
}

template <typename KernelT>
cudaError_t ensure_smem(KernelT kernel, uint32_t bytes, bool (&done)[64]) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !done[dev]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
        if (dev < 64) done[dev] = true;
    }
    return cudaSuccess;
}

template <typename T, int K>
cudaError_t launch_t(const Problem& p, const BackwardArgs& ga, const float* wt, float* ws_a, float* ws_dl,
                     int* d_status, int num_sms, cudaStream_t stream) {
    using C_ = Cfg<T, K>;
    static bool done_a[64] = {}, done_b[64] = {}, done_c[64] = {};
    cudaError_t e = ensure_smem(bwd_point_kernel<T, K>, PointCfg<T, K>::total, done_a);
    if (e == cudaSuccess) e = ensure_smem(bwd_gather_kernel<T, K>, GatherCfg<T, K>::total, done_b);
    if (e == cudaSuccess) e = ensure_smem(bwd_weight_kernel<T, K>, WeightCfg<T, K>::total, done_c);
    if (e != cudaSuccess) return e;
    BwdParams P;
    P.wt = wt; P.bias = p.bias;
    P.dq = ga.dq; P.dk = ga.dk; P.dv = ga.dv; P.dwk = ga.dwk; P.dwv = ga.dwv; P.dbias = ga.dbias;
    P.ws_a = ws_a; P.ws_dl = ws_dl; P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.tiles_x = (p.W + kTW - 1) / kTW;
    P.tiles_y = (p.H + C_::TH - 1) / C_::TH;
    P.scale = 1.f / sqrtf((float)kHeadDim);
    const int Ctot = p.heads * kHeadDim;
    const int cpp = 64 / (int)sizeof(T);
    const int es = (int)sizeof(T);
    CUtensorMap mq, mk, mv, mg, mqh, mgh;
    if (!make_tile_map(&mq, p.q, es, p.B, p.H, p.W, Ctot, cpp, kTW, C_::TH) ||
        !make_tile_map(&mg, ga.dout, es, p.B, p.H, p.W, Ctot, cpp, kTW, C_::TH) ||
        !make_tile_map(&mk, p.k, es, p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH) ||
        !make_tile_map(&mv, p.v, es, p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH) ||
        !make_tile_map(&mqh, p.q, es, p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH) ||
        !make_tile_map(&mgh, ga.dout, es, p.B, p.H, p.W, Ctot, cpp, C_::HW, C_::HH))
        return cudaErrorInvalidValue;
    const long long tiles_per_head = (long long)P.tiles_x * P.tiles_y * p.B;
    const long long ctas = tiles_per_head * p.heads;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    bwd_point_kernel<T, K><<<(unsigned)ctas, C_::threads, PointCfg<T, K>::total, stream>>>(mq, mk, mv, mg, P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    bwd_gather_kernel<T, K><<<(unsigned)ctas, C_::threads, GatherCfg<T, K>::total, stream>>>(mqh, mgh, P);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    long long per_head = (2LL * num_sms + p.heads - 1) / p.heads;            // persistent CTAs of the weight kernel
    if (per_head > tiles_per_head) per_head = tiles_per_head;
    if (per_head < 1) per_head = 1;
    bwd_weight_kernel<T, K><<<(unsigned)(per_head * p.heads), C_::threads, WeightCfg<T, K>::total, stream>>>(mq, mk, mv, mg, P);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_k(const Problem& p, const BackwardArgs& ga, const float* wt, float* ws_a, float* ws_dl,
                     int* d_status, int num_sms, cudaStream_t stream) {
    switch (p.ksize) {
        case 1: return launch_t<T, 1>(p, ga, wt, ws_a, ws_dl, d_status, num_sms, stream);
        case 3: return launch_t<T, 3>(p, ga, wt, ws_a, ws_dl, d_status, num_sms, stream);
        default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace

bool backward_supports(int head_dim, int ksize) {
    return head_dim == kHeadDim && (ksize == 1 || ksize == 3) && tensor_map_available();
}

size_t backward_workspace_bytes(int B, int H, int W, int heads, int ksize) {
    return 2 * (size_t)B * H * W * heads * ksize * ksize * sizeof(float);
}

// `wt`: transposed weights as launch_strip_prep writes them; `ws`: backward_workspace_bytes of scratch.
// The weight and bias gradients must be zero when the first kernel starts (the caller of this function
// clears them on the same stream).
cudaError_t launch_backward(const Problem& p, const BackwardArgs& ga, const void* wt, void* ws, int* d_status,
                            int num_sms, cudaStream_t stream) {
    float* ws_a = static_cast<float*>(ws);
    float* ws_dl = ws_a + (size_t)p.B * p.H * p.W * p.heads * p.ksize * p.ksize;
    const float* w = static_cast<const float*>(wt);
    return p.dtype == SLIDE_ATTN_BF16 ? launch_k<__nv_bfloat16>(p, ga, w, ws_a, ws_dl, d_status, num_sms, stream)
                                      : launch_k<float>(p, ga, w, ws_a, ws_dl, d_status, num_sms, stream);
}

}  // namespace slide_attn
