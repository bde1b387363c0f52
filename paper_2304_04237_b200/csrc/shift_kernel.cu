// Fixed-shift fast path (Sec. 4.2, Eq. 8-13): when both depthwise kernels are exactly the one-hot
// shift kernels of Eq. 11 (no deformed-shift term), slot s of a query pixel IS the key / value at
// window offset s, so the forward is plain k x k local attention with zero padding (Eq. 2 over
// r_q = the pixel's own neighbourhood; padded slots keep key 0, value 0 and their softmax mass):
//
//   l[s]     = (q[p] . k[p + off(s)]) / sqrt(d) + bias[s]
//   a        = softmax_s(l)
//   out[p,c] = sum_s a[s] v[p + off(s), c]
//
// 2 k^2 multiply-adds per pixel-channel instead of 2 k^4 + 2 k^2: for small windows the pass is bound by
// HBM, so it runs on the CUDA cores straight off a halo tile.
//
// One CTA = one head of a 4 x 32 pixel tile (four warps; several CTAs share an SM, so one CTA's loads
// overlap another's arithmetic).  The K and V tile + floor(k/2) halo and the q tile come in
// by TMA (out-of-map elements zero-filled: that IS the padding) as "planes" of 64 bytes of channels per
// pixel (bf16: one plane of 32 channels; fp32: two planes of 16), so that a quad of lanes reads one
// pixel's plane as four 16-byte pieces and a warp-wide load covers 512 contiguous bytes.  A warp owns 8
// columns x 4 rows; lane (g, tig) = column g, channels of piece tig (eight per lane).  For every window
// column dx the warp walks the 4 + k - 1 halo rows of that column once: each row vector serves every
// pixel of the strip whose window holds it.  The softmax runs online over the window columns (running
// maximum, sum and accumulator per pixel), so registers do not grow with k^2.
#include "tile_common.cuh"

namespace slide_attn {

namespace {

using namespace tile;
using ShiftParams = TileParams;

template <typename T, int K>
__global__ void __launch_bounds__(Cfg<T, K>::threads, (sizeof(T) == 2 && K <= 3) ? 6 : 4)
shift_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
             const __grid_constant__ CUtensorMap map_v, const ShiftParams P)
{
    using C_ = Cfg<T, K>;
    constexpr int R = K / 2;
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
    for (int i = threadIdx.x; i < K * K; i += C_::threads) s_bias[i] = P.bias ? P.bias[h * K * K + i] * kLog2e : 0.f;
    __syncthreads();
    if (!mbar_wait(bar, 0)) {                                  // bounded: about two seconds
        if (lane == 0) atomicExch(P.status, 1);
        return;
    }

    const int wx = warp % (kTW / 8), wy = warp / (kTW / 8);
    const int col = wx * 8 + g, row0 = wy * kR;                  // this lane's pixel column, first pixel row
    const unsigned char* sK = smem + C_::k_off;
    const unsigned char* sV = smem + C_::v_off;
    const unsigned char* sQ = smem + C_::q_off;

    // Within a quad, lane tig also OWNS pixel row tig of the strip: the partial dot products of the
    // four lanes are summed so that each lane ends up with the k logits of its own pixel (a
    // transpose-reduce), the softmax bookkeeping is done once per pixel, and the weights go back to
    // all four lanes for the value side.
    static_assert(kR == 4, "one pixel row per lane of a quad");
    const int qbase = lane & ~3;
    typename Piece<T>::Raw qr[kR];
#pragma unroll
    for (int r = 0; r < kR; ++r) qr[r] = Piece<T>::load(sQ, C_::q_plane, (uint32_t)((row0 + r) * kTW + col), tig);
    float m = -INFINITY, sum = 0.f;                              // of pixel row tig
    float acc[kR][8];
#pragma unroll
    for (int r = 0; r < kR; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;

#pragma unroll 1
    for (int dx = 0; dx < K; ++dx) {
        // partial logits of window column dx: halo row j serves pixel r at window row dy = j - r
        float p[kR][K];
#pragma unroll
        for (int j = 0; j < kR + K - 1; ++j) {
            const typename Piece<T>::Raw kv = Piece<T>::load(sK, C_::halo_plane, (uint32_t)((row0 + j) * C_::HW + col + dx), tig);
#pragma unroll
            for (int r = 0; r < kR; ++r) {
                const int dy = j - r;
                if (dy >= 0 && dy < K) p[r][dy] = Piece<T>::dot(qr[r], kv);
            }
        }
        // transpose-reduce over the quad: afterwards l[dy] is the full dot product of pixel row tig
        float l[K];
#pragma unroll
        for (int dy = 0; dy < K; ++dy) {
            const bool up = (tig & 2) != 0;
            const float s0 = up ? p[0][dy] : p[2][dy], s1 = up ? p[1][dy] : p[3][dy];
            const float k0 = (up ? p[2][dy] : p[0][dy]) + __shfl_xor_sync(0xffffffffu, s0, 2);
            const float k1 = (up ? p[3][dy] : p[1][dy]) + __shfl_xor_sync(0xffffffffu, s1, 2);
            const bool odd = (tig & 1) != 0;
            l[dy] = (odd ? k1 : k0) + __shfl_xor_sync(0xffffffffu, odd ? k0 : k1, 1);
        }
        float cm = -INFINITY;
#pragma unroll
        for (int dy = 0; dy < K; ++dy) { l[dy] = fmaf(l[dy], P.scale_log2e, s_bias[dy * K + dx]); cm = fmaxf(cm, l[dy]); }
        const float mn = fmaxf(m, cm);
        const float corr = fast_exp2(m - mn);                    // 0 for the first column (m = -inf)
        m = mn;
        sum *= corr;
#pragma unroll
        for (int dy = 0; dy < K; ++dy) { l[dy] = fast_exp2(l[dy] - mn); sum += l[dy]; }
        // weights and rescale factors of all four pixel rows, in every lane of the quad
        float e[kR][K], cr[kR];
#pragma unroll
        for (int r = 0; r < kR; ++r) {
            cr[r] = __shfl_sync(0xffffffffu, corr, qbase + r);
#pragma unroll
            for (int dy = 0; dy < K; ++dy) e[r][dy] = __shfl_sync(0xffffffffu, l[dy], qbase + r);
        }
#pragma unroll
        for (int r = 0; r < kR; ++r)
#pragma unroll
            for (int c = 0; c < 8; c += 2) fmul2(acc[r][c], acc[r][c + 1], cr[r], cr[r]);
#pragma unroll
        for (int j = 0; j < kR + K - 1; ++j) {
            float vv[8];
            Piece<T>::widen(Piece<T>::load(sV, C_::halo_plane, (uint32_t)((row0 + j) * C_::HW + col + dx), tig), vv);
#pragma unroll
            for (int r = 0; r < kR; ++r) {
                const int dy = j - r;
                if (dy >= 0 && dy < K) {
                    const float w = e[r][dy];
#pragma unroll
                    for (int c = 0; c < 8; c += 2) ffma2(acc[r][c], acc[r][c + 1], w, w, vv[c], vv[c + 1]);
                }
            }
        }
    }
    const float my_inv = 1.f / sum;
    float invs[kR];
#pragma unroll
    for (int r = 0; r < kR; ++r) invs[r] = __shfl_sync(0xffffffffu, my_inv, qbase + r);

    const int x = x0 + col;
    const int Ctot = P.heads * kHeadDim;
#pragma unroll
    for (int r = 0; r < kR; ++r) {
        const int y = y0 + row0 + r;
        if (x < P.W && y < P.H) {
            const float inv = invs[r];
            const size_t base = ((size_t)(b * P.H + y) * P.W + x) * Ctot + h * kHeadDim;
            if constexpr (sizeof(T) == 2) {
                uint4 o;
                o.x = pack_bf16(acc[r][0] * inv, acc[r][1] * inv); o.y = pack_bf16(acc[r][2] * inv, acc[r][3] * inv);
                o.z = pack_bf16(acc[r][4] * inv, acc[r][5] * inv); o.w = pack_bf16(acc[r][6] * inv, acc[r][7] * inv);
                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(P.out) + base + tig * 8) = o;
            } else {
                float* op = static_cast<float*>(P.out) + base;
                *reinterpret_cast<float4*>(op + tig * 4) = make_float4(acc[r][0] * inv, acc[r][1] * inv, acc[r][2] * inv, acc[r][3] * inv);
                *reinterpret_cast<float4*>(op + 16 + tig * 4) = make_float4(acc[r][4] * inv, acc[r][5] * inv, acc[r][6] * inv, acc[r][7] * inv);
            }
        }
    }
}

// Sets the status word to 2 if any weight differs from the one-hot shift kernel w[c][s][t] = [s == t].
__global__ void shift_check_kernel(const float* __restrict__ wk, const float* __restrict__ wv, long long n_per, int k2, int* status)
{
    grid_launch_dependents();        // the fixed-shift kernel does not read this kernel's result
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < 2 * n_per; i += (long long)gridDim.x * blockDim.x) {
        const long long j = i < n_per ? i : i - n_per;
        const int st = (int)(j % ((long long)k2 * k2));
        const float want = (st / k2 == st % k2) ? 1.f : 0.f;
        const float got = i < n_per ? wk[j] : wv[j];
        bad |= !(got == want);
    }
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicExch(status, 2);
}

template <typename T, int K>
cudaError_t launch_t(const Problem& p, int* d_status, cudaStream_t stream) {
    using C_ = Cfg<T, K>;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && !configured[dev]) {
        e = cudaFuncSetAttribute(shift_kernel<T, K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C_::total);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    } else if (dev >= 64) {
        e = cudaFuncSetAttribute(shift_kernel<T, K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C_::total);
        if (e != cudaSuccess) return e;
    }
    ShiftParams P;
    P.wt = nullptr; P.bias = p.bias; P.out = p.out; P.status = d_status;
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
    // programmatic stream serialisation: the kernel may run beside the weight check launched just
    // before it (it does not read the check's result; both only ever set the status word)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(C_::threads);
    cfg.dynamicSmemBytes = C_::total;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, shift_kernel<T, K>, mq, mk, mv, P);
}

template <typename T>
cudaError_t launch_k(const Problem& p, int* d_status, cudaStream_t stream) {
    switch (p.ksize) {
        case 1: return launch_t<T, 1>(p, d_status, stream);
        case 3: return launch_t<T, 3>(p, d_status, stream);
        case 5: return launch_t<T, 5>(p, d_status, stream);
        case 7: return launch_t<T, 7>(p, d_status, stream);
        case 9: return launch_t<T, 9>(p, d_status, stream);
        default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace

bool shift_supports(int head_dim, int ksize) {
    return head_dim == kHeadDim && (ksize & 1) && ksize >= 1 && ksize <= 9 && tensor_map_available();
}

cudaError_t launch_shift_check(const Problem& p, int* d_status, cudaStream_t stream) {
    const int k2 = p.ksize * p.ksize;
    const long long n_per = (long long)p.heads * p.head_dim * k2 * k2;
    const int blocks = (int)((2 * n_per + 255) / 256 < 1184 ? (2 * n_per + 255) / 256 : 1184);
    shift_check_kernel<<<blocks, 256, 0, stream>>>(p.wk, p.wv, n_per, k2, d_status);
    return cudaGetLastError();
}

cudaError_t launch_shift(const Problem& p, int* d_status, cudaStream_t stream) {
    return p.dtype == SLIDE_ATTN_BF16 ? launch_k<__nv_bfloat16>(p, d_status, stream) : launch_k<float>(p, d_status, stream);
}

}  // namespace slide_attn
