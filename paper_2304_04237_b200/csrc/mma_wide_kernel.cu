// MMA_WIDE variant: deformed (general) depthwise weights with LARGE windows on tensor cores (the
// paper's stated limitation, App. E-F: k > 3 costs "a huge increase on the inference time"): bf16,
// head_dim 32, k = 5, 7, 9 (k = 3 compiles too and serves as a cross-check).
//
// Arithmetic (Eq. 2 with Eq. 12 inside; w = E + D, E the one-hot shift of Eq. 11, D the remainder):
//   P[p,(t,c)]  = q[p,c] k[p+off(t),c]                    packed bf16 multiply, formed in registers as
//                                                          the A fragment of mma.sync.m16n8k16
//   Ld[p,s]    += sum_c P[p,(t,c)] D_k[c,s,t]             k^2 taps x 2 k-steps x k^2/8 n-tiles
//   Lp[p,t]    += sum_c P[p,(t,c)]                        one more MMA per k-step against a 0/1 fragment:
//                                                          the plain q.k sum of tap t, exact products
//   logit[s]    = (Ld[s] + Lp[s]) scale + bias[s];  e = exp2(logit - max)    (quad shuffles)
//   A'[p,(t,c)] = e[p,t] + sum_s e_hi[p,s] D_v[c,s,t]     accumulator initialised to the exact fp32 e[p,t];
//                                                          the logits' C fragments ARE the A fragments
//   out[p,c]    = (sum_t A'[p,t,c] v[p+off(t),c]) / sum_s e[p,s]             packed fp32 FMAs
// 2 k^4 multiply-adds per pixel-channel go to the tensor cores; the CUDA cores keep 2 k^2.
//
// One CTA = one head of a 4 x 32 pixel tile: K / V halo tiles and the q tile by TMA (64-byte channel
// planes, zero fill = the padding); eight compute warps, each 2 rows x 8 columns = the 16 rows of an
// MMA (lane (g, tig): column g, both rows, channels 8 tig .. 8 tig + 7).  The weights do not fit on
// chip for k >= 5 (2 x 32 k^4 bf16 per head: 100 KB at k = 5, 950 KB at k = 9), so a ninth warp
// streams them from L2 tap by tap through a four-stage ring of bulk copies, in the register-fragment
// order a prep kernel wrote them in: first the k^2 key-side chunks, then the k^2 value-side chunks.
// Every wait is bounded and sets the status word.
//
// Measured and not kept: two M tiles per warp (a weight fragment then feeds two MMAs, but half as many
// warps with twice the registers ran 1.1-1.9x slower); 16-byte loads of two n-tiles' fragments at once
// (within +-8 % of the 8-byte form).
#include "tile_common.cuh"

namespace slide_attn {

namespace {

using namespace tile;

template <int K>
struct Wide {
    static constexpr int K2 = K * K;
    static constexpr int KS = (K2 + 15) / 16;        // k-steps of the value MMA (slots, 16 per step)
    static constexpr int NT = 2 * KS;                // n-tiles of 8 slots on the key side (covers 16 KS slots)
    static constexpr int chunk_bytes = 2 * NT * 256; // one tap: key side [2 kh][NT][32 lanes][8 B] = value side [KS][4][32][8 B]
    static constexpr int stages = 4;
    using C_ = Cfg<__nv_bfloat16, K>;
    static constexpr uint32_t ring_off = C_::bar_off + 128;                       // barriers: tile, full[4], empty[4]
    static constexpr uint32_t total = ring_off + stages * chunk_bytes + 128;
    static constexpr int threads = C_::threads * 2 + 32;                          // eight compute warps + the streaming warp
};

struct WideParams {
    const unsigned char* frag;       // [head][2 K2 chunks][chunk_bytes]
    const float* bias;
    __nv_bfloat16* out;
    int* status;
    int B, H, W, heads;
    int tiles_x, tiles_y;
    float scale_log2e;
};

// Prep: fp32 [C][slot][tap] -> bf16 B fragments of mma.sync.m16n8k16 (b0 = rows 2 tig, 2 tig + 1 of
// column g; b1 = rows 2 tig + 8, 2 tig + 9), one 8-byte item per (chunk, unit, lane).
//   key chunk t, unit (kh, j): row kappa = 2 tig' + e + 8 j' of k-step kh is channel 8 tig' + 4 kh + 2 j' + e
//                              (the order in which a lane's 16-byte piece fills the A fragment);
//                              column g of n-tile j is slot 8 j + g; value D_k[c][slot][t]
//   value chunk t, unit (ks, jc): row kappa of k-step ks is slot 16 ks + kappa; column g' of n-tile jc is
//                              channel 8 (g' >> 1) + 2 jc + (g' & 1); value D_v[c][slot][t]
template <int K>
__global__ void __launch_bounds__(256)
mma_wide_prep_kernel(const float* __restrict__ wk, const float* __restrict__ wv, unsigned char* __restrict__ frag, int heads)
{
    using Wd = Wide<K>;
    constexpr int K2 = Wd::K2, NT = Wd::NT, KS = Wd::KS;
    const long long items = (long long)heads * 2 * K2 * 2 * NT * 32;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < items; i += (long long)gridDim.x * blockDim.x) {
        const int lane = (int)(i & 31);
        long long r = i >> 5;
        const int unit = (int)(r % (2 * NT)); r /= 2 * NT;
        const int chunk = (int)(r % (2 * K2));
        const int h = (int)(r / (2 * K2));
        const int g = lane >> 2, tig = lane & 3;
        float val[4];
        if (chunk < K2) {
            const int t = chunk, kh = unit / NT, j = unit % NT;
            const int s = 8 * j + g;
#pragma unroll
            for (int x = 0; x < 4; ++x) {                      // x = 2 j' + e
                const int c = h * kHeadDim + 8 * tig + 4 * kh + x;
                val[x] = s < K2 ? wk[((size_t)c * K2 + s) * K2 + t] - (s == t ? 1.f : 0.f) : 0.f;
            }
        } else {
            const int t = chunk - K2, ks = unit / 4, jc = unit % 4;
            const int c = h * kHeadDim + 8 * (g >> 1) + 2 * jc + (g & 1);
#pragma unroll
            for (int x = 0; x < 4; ++x) {                      // x = 2 j' + e: slot 16 ks + 2 tig + e + 8 j'
                const int s = 16 * ks + 2 * tig + (x & 1) + 8 * (x >> 1);
                val[x] = (unit < 4 * KS && s < K2) ? wv[((size_t)c * K2 + s) * K2 + t] - (s == t ? 1.f : 0.f) : 0.f;
            }
        }
        *reinterpret_cast<uint2*>(frag + (size_t)i * 8) = make_uint2(pack_bf16(val[0], val[1]), pack_bf16(val[2], val[3]));
    }
}

template <int K>
__global__ void __launch_bounds__(Wide<K>::threads)
mma_wide_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const WideParams P)
{
    using T = __nv_bfloat16;
    using C_ = Cfg<T, K>;
    using Wd = Wide<K>;
    constexpr int R = K / 2, K2 = Wd::K2, NT = Wd::NT, KS = Wd::KS, ST = Wd::stages;
    constexpr int NTS = (K2 + 7) / 8;                            // n-tiles that hold real slots
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t bar0 = smem_u32(smem + C_::bar_off);
    const uint32_t bar_tile = bar0;
    auto bar_full = [&](int s) { return bar0 + 8u * (uint32_t)(1 + s); };
    auto bar_empty = [&](int s) { return bar0 + 8u * (uint32_t)(1 + ST + s); };
    float* s_bias = reinterpret_cast<float*>(smem + C_::bias_off);
    const unsigned char* ring = smem + Wd::ring_off;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int h = blockIdx.x % P.heads;
    int rest = blockIdx.x / P.heads;
    const int tx = rest % P.tiles_x; rest /= P.tiles_x;
    const int ty = rest % P.tiles_y;
    const int b = rest / P.tiles_y;
    const int x0 = tx * kTW, y0 = ty * C_::TH;
    constexpr int kCWarps = 8;

    if (threadIdx.x == 0) {
        mbar_init_only(bar_tile, 1);
        for (int s = 0; s < ST; ++s) { mbar_init_only(bar_full(s), 1); mbar_init_only(bar_empty(s), kCWarps); }
        mbar_init_fence();
        mbar_expect_tx(bar_tile, C_::tx_bytes);
        const int c0 = h * kHeadDim;
        tma_load_4d(smem_u32(smem + C_::k_off), &map_k, bar_tile, c0, x0 - R, y0 - R, b);
        tma_load_4d(smem_u32(smem + C_::v_off), &map_v, bar_tile, c0, x0 - R, y0 - R, b);
        tma_load_4d(smem_u32(smem + C_::q_off), &map_q, bar_tile, c0, x0, y0, b);
    }
    for (int i = threadIdx.x; i < K2; i += Wd::threads) s_bias[i] = P.bias ? P.bias[h * K2 + i] * kLog2e : 0.f;
    __syncthreads();

    if (warp == kCWarps) {
        // ---- streaming warp: 2 K2 weight chunks of this head through the ring -------------------------
        if (lane == 0) {
            const unsigned char* src = P.frag + (size_t)h * 2 * K2 * Wd::chunk_bytes;
            bool ok = true;
            for (int i = 0; i < 2 * K2; ++i) {
                const int s = i % ST;
                if (i >= ST && !mbar_wait(bar_empty(s), (uint32_t)(i / ST - 1) & 1u)) { ok = false; break; }
                mbar_expect_tx(bar_full(s), Wd::chunk_bytes);
                bulk_load_1d(smem_u32(ring + s * Wd::chunk_bytes), src + (size_t)i * Wd::chunk_bytes, Wd::chunk_bytes, bar_full(s));
            }
            if (!ok) atomicExch(P.status, 1);
        }
        return;
    }

    // ---- compute warps ---------------------------------------------------------------------------------
    bool ok = __all_sync(0xffffffffu, mbar_wait(bar_tile, 0) ? 1 : 0) != 0;
    const int wx = warp & 3, wy = warp >> 2;                       // column group, row pair
    const int col = wx * 8 + g, row0 = 2 * wy;
    const unsigned char* sK = smem + C_::k_off;
    const unsigned char* sV = smem + C_::v_off;
    const unsigned char* sQ = smem + C_::q_off;
    auto piece = [&](const unsigned char* tile, int pix) { return *reinterpret_cast<const uint4*>(tile + (uint32_t)pix * 64u + tig * 16u); };

    uint4 qa = make_uint4(0, 0, 0, 0), qb = qa;
    if (ok) { qa = piece(sQ, row0 * kTW + col); qb = piece(sQ, (row0 + 1) * kTW + col); }

    float ld[NT][4], lp[NTS][4];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int x = 0; x < 4; ++x) ld[j][x] = 0.f;
#pragma unroll
    for (int j = 0; j < NTS; ++j)
#pragma unroll
        for (int x = 0; x < 4; ++x) lp[j][x] = 0.f;

    int chunk = 0;                                                  // position in the stream of 2 K2 chunks
#pragma unroll
    for (int t = 0; t < K2; ++t, ++chunk) {
        const int dy = t / K, dx = t % K;
        const int s = chunk % ST;
        if (ok && !__all_sync(0xffffffffu, mbar_wait(bar_full(s), (uint32_t)(chunk / ST) & 1u) ? 1 : 0)) ok = false;
        if (ok) {
            const uint4 ka = piece(sK, (row0 + dy) * C_::HW + col + dx), kb = piece(sK, (row0 + 1 + dy) * C_::HW + col + dx);
            const uint32_t pa[4] = {hmul2_bf16(qa.x, ka.x), hmul2_bf16(qa.y, ka.y), hmul2_bf16(qa.z, ka.z), hmul2_bf16(qa.w, ka.w)};
            const uint32_t pb[4] = {hmul2_bf16(qb.x, kb.x), hmul2_bf16(qb.y, kb.y), hmul2_bf16(qb.z, kb.z), hmul2_bf16(qb.w, kb.w)};
            const unsigned char* bsrc = ring + s * Wd::chunk_bytes + lane * 8;
            const uint32_t ones = (g == (t & 7)) ? kOnesBf16x2 : 0u;
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                const uint32_t a[4] = {pa[2 * kh], pb[2 * kh], pa[2 * kh + 1], pb[2 * kh + 1]};
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const uint2 bf = *reinterpret_cast<const uint2*>(bsrc + (kh * NT + j) * 256);
                    mma_bf16(ld[j], a, bf.x, bf.y);
                }
                mma_bf16(lp[t >> 3], a, ones, ones);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty(s));
    }

    // ---- softmax over the k^2 slots: a quad holds one pixel's logits (lane tig: slots 8 j + 2 tig, + 1) ---
    float ev[2][NT][2];                                             // [pixel row][n-tile][slot parity]
    float inv[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int s = 8 * j + 2 * tig + e;
                float v = -INFINITY;
                if (j < NTS && s < K2) v = fmaf(ld[j][2 * r + e] + lp[j][2 * r + e], P.scale_log2e, s_bias[s]);
                ev[r][j][e] = v;
                m = fmaxf(m, v);
            }
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        float z = 0.f;
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) { ev[r][j][e] = fast_exp2(ev[r][j][e] - m); z += ev[r][j][e]; }   // exp2(-inf) = 0 for the padding slots
        z += __shfl_xor_sync(0xffffffffu, z, 1);
        z += __shfl_xor_sync(0xffffffffu, z, 2);
        inv[r] = 1.f / z;
    }
    // the logits' C fragments are the A fragments of the value MMA (bf16: the deformed part is small)
    uint32_t ah[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        ah[ks][0] = pack_bf16(ev[0][2 * ks][0], ev[0][2 * ks][1]);
        ah[ks][1] = pack_bf16(ev[1][2 * ks][0], ev[1][2 * ks][1]);
        ah[ks][2] = pack_bf16(ev[0][2 * ks + 1][0], ev[0][2 * ks + 1][1]);
        ah[ks][3] = pack_bf16(ev[1][2 * ks + 1][0], ev[1][2 * ks + 1][1]);
    }

    float oa[8], ob[8];                                              // the two pixel rows, channels 8 tig ..
#pragma unroll
    for (int c = 0; c < 8; ++c) { oa[c] = 0.f; ob[c] = 0.f; }
#pragma unroll
    for (int t = 0; t < K2; ++t, ++chunk) {
        const int dy = t / K, dx = t % K;
        const int s = chunk % ST;
        if (ok && !__all_sync(0xffffffffu, mbar_wait(bar_full(s), (uint32_t)(chunk / ST) & 1u) ? 1 : 0)) ok = false;
        // e[p][t] of the two pixels: slot t lives in quad lane (t % 8) / 2, n-tile t / 8, parity t % 2
        const float ea = __shfl_sync(0xffffffffu, ev[0][t >> 3][t & 1], (lane & ~3) | ((t & 7) >> 1));
        const float eb = __shfl_sync(0xffffffffu, ev[1][t >> 3][t & 1], (lane & ~3) | ((t & 7) >> 1));
        if (ok) {
            float cf[4][4];
#pragma unroll
            for (int jc = 0; jc < 4; ++jc) { cf[jc][0] = ea; cf[jc][1] = ea; cf[jc][2] = eb; cf[jc][3] = eb; }
            const unsigned char* bsrc = ring + s * Wd::chunk_bytes + lane * 8;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                for (int jc = 0; jc < 4; ++jc) {
                    const uint2 bf = *reinterpret_cast<const uint2*>(bsrc + (ks * 4 + jc) * 256);
                    mma_bf16(cf[jc], ah[ks], bf.x, bf.y);
                }
            const uint4 va = piece(sV, (row0 + dy) * C_::HW + col + dx), vb = piece(sV, (row0 + 1 + dy) * C_::HW + col + dx);
            const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
            for (int jc = 0; jc < 4; ++jc) {                       // channels 8 tig + 2 jc, + 1 = word jc of the piece
                ffma2(oa[2 * jc], oa[2 * jc + 1], cf[jc][0], cf[jc][1], bf16_lo(wa[jc]), bf16_hi(wa[jc]));
                ffma2(ob[2 * jc], ob[2 * jc + 1], cf[jc][2], cf[jc][3], bf16_lo(wb[jc]), bf16_hi(wb[jc]));
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty(s));
    }

    if (!ok) { if (lane == 0) atomicExch(P.status, 1); return; }
    const int x = x0 + col, y = y0 + row0;
    const int Ctot = P.heads * kHeadDim;
    if (x < P.W) {
        if (y < P.H) {
            uint4 o;
            o.x = pack_bf16(oa[0] * inv[0], oa[1] * inv[0]); o.y = pack_bf16(oa[2] * inv[0], oa[3] * inv[0]);
            o.z = pack_bf16(oa[4] * inv[0], oa[5] * inv[0]); o.w = pack_bf16(oa[6] * inv[0], oa[7] * inv[0]);
            *reinterpret_cast<uint4*>(P.out + ((size_t)(b * P.H + y) * P.W + x) * Ctot + h * kHeadDim + tig * 8) = o;
        }
        if (y + 1 < P.H) {
            uint4 o;
            o.x = pack_bf16(ob[0] * inv[1], ob[1] * inv[1]); o.y = pack_bf16(ob[2] * inv[1], ob[3] * inv[1]);
            o.z = pack_bf16(ob[4] * inv[1], ob[5] * inv[1]); o.w = pack_bf16(ob[6] * inv[1], ob[7] * inv[1]);
            *reinterpret_cast<uint4*>(P.out + ((size_t)(b * P.H + y + 1) * P.W + x) * Ctot + h * kHeadDim + tig * 8) = o;
        }
    }
}

template <int K>
cudaError_t launch_t(const Problem& p, void* workspace, int* d_status, cudaStream_t stream) {
    using Wd = Wide<K>;
    using C_ = Cfg<__nv_bfloat16, K>;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(mma_wide_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Wd::total);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured[dev] = true;
    }
    const long long items = (long long)p.heads * 2 * Wd::K2 * 2 * Wd::NT * 32;
    long long pblocks = (items + 255) / 256;
    if (pblocks > 2368) pblocks = 2368;
    mma_wide_prep_kernel<K><<<(unsigned)pblocks, 256, 0, stream>>>(p.wk, p.wv, static_cast<unsigned char*>(workspace), p.heads);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    WideParams P;
    P.frag = static_cast<const unsigned char*>(workspace);
    P.bias = p.bias; P.out = static_cast<__nv_bfloat16*>(p.out); P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.tiles_x = (p.W + kTW - 1) / kTW;
    P.tiles_y = (p.H + C_::TH - 1) / C_::TH;
    P.scale_log2e = kLog2e / sqrtf((float)kHeadDim);
    const int Ctot = p.heads * kHeadDim;
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, p.q, 2, p.B, p.H, p.W, Ctot, kHeadDim, kTW, C_::TH) ||
        !make_tile_map(&mk, p.k, 2, p.B, p.H, p.W, Ctot, kHeadDim, C_::HW, C_::HH) ||
        !make_tile_map(&mv, p.v, 2, p.B, p.H, p.W, Ctot, kHeadDim, C_::HW, C_::HH))
        return cudaErrorInvalidValue;
    const long long ctas = (long long)P.tiles_x * P.tiles_y * p.B * p.heads;
    if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    mma_wide_kernel<K><<<(unsigned)ctas, Wd::threads, Wd::total, stream>>>(mq, mk, mv, P);
    return cudaGetLastError();
}

}  // namespace

bool mma_wide_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && (ksize == 3 || ksize == 5 || ksize == 7 || ksize == 9) &&
           tensor_map_available();
}

size_t mma_wide_workspace_bytes(int heads, int ksize) {
    switch (ksize) {
        case 3: return (size_t)heads * 2 * 9 * Wide<3>::chunk_bytes;
        case 5: return (size_t)heads * 2 * 25 * Wide<5>::chunk_bytes;
        case 7: return (size_t)heads * 2 * 49 * Wide<7>::chunk_bytes;
        case 9: return (size_t)heads * 2 * 81 * Wide<9>::chunk_bytes;
        default: return 0;
    }
}

// Prep launch (weights -> fragment-ordered chunks in `workspace`) followed by the fused kernel.
cudaError_t launch_mma_wide(const Problem& p, void* workspace, int* d_status, cudaStream_t stream) {
    switch (p.ksize) {
        case 3: return launch_t<3>(p, workspace, d_status, stream);
        case 5: return launch_t<5>(p, workspace, d_status, stream);
        case 7: return launch_t<7>(p, workspace, d_status, stream);
        case 9: return launch_t<9>(p, workspace, d_status, stream);
        default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace slide_attn
