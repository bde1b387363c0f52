// MMA variant (bf16, head_dim 32, k = 3): the deformed-shift contraction on tensor cores.
//
// The merged kernels are split as w = E + D, E the one-hot shift of Eq. 11 (w[c,s,t] = 1 iff
// t == s) and D the remainder (the learned deformed shift of Sec. 4.3; any w works, D is just
// w - E).  With P[p,t,c] = q[p,c] * k[p+off(t),c]:
//
//   logit[p,s] = sum_{t,c} P[p,t,c] * (D_k[c,s,t] + [t == s])            (Eq. 2 with Eq. 12 inside)
//   A'[p,t,c]  = e[p,t] + sum_s e[p,s] * D_v[c,s,t],   e = exp(logit - max)
//   out[p,c]   = (sum_t A'[p,t,c] * v[p+off(t),c]) / sum_s e[p,s]
//
// Both sums over (t,c) resp. s are dense contractions shared by all pixels of a head, so they run
// as mma.sync.m16n8k16 (bf16 operands, fp32 accumulate).  The one-hot part of the key side rides
// in spare columns of the padded slot dimension (9 slots -> 16 columns), so its weight 1.0 is
// exact; on the value side it is the exact fp32 initial value of the accumulator.
//
// One CTA handles one head of a TH x TW pixel tile.  The tile plus its one-pixel halo of K and V
// (32 channels = 64 B per pixel) is fetched by two TMA loads whose out-of-map elements are filled
// with zeros: that fill is the zero padding of the convolution.  A warp works on "units" of
// 4 rows x 8 columns: lane (g, tig) = (lane/4, lane%4) owns column g, all four rows, channels
// 8*tig .. 8*tig+7, i.e. rows g and g+8 of two 16-row MMA tiles (rows 0,1 and rows 2,3).
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

namespace {

constexpr int kHeadDim = 32;
constexpr int kWarps = 8;
constexpr int kFragWordsPerHead = 4608;        // 2304 (key side) + 2304 (value side) uint32
constexpr uint32_t kOnes = kOnesBf16x2;

// ---------------------------------------------------------------------------------------------
// Weight re-layout: fp32 [C][9][9] -> bf16x2 words in the order the MMA B-fragments are loaded.
//
// Key side, word (t, ks, lane, i): n-tile nt = i/2, register r = i%2.  B is [k = 16 channels] x
// [n = 8 columns]; a lane holds column n = g and rows (2*tig, 2*tig+1) (+8 for r = 1).  Row kc of
// k-step ks is channel 8*((kc%8)/2) + 4*ks + 2*(kc/8) + kc%2 of the head, which is where the A
// operand (built from one 16-byte shared-memory load per pixel) has that channel.
//   n-tile 0, column n: slot n,  value D_k[c][n][t]
//   n-tile 1, column 0: slot 8,  value D_k[c][8][t];  column 1: [t == 0];  column n >= 2: [t == n]
// (taps 1 and 8 get their one-hot column from a constant third n-tile inside the main kernel).
//
// Value side, word (t, jp, lane, i): n-tile j = 2*jp + i/2, register r = i%2.  B is [k = 16 slots]
// x [n = 8 channels]; column n is channel 8*(n/2) + 2*j + n%2; rows 0..8 are the slots, 9..15 zero.
// ---------------------------------------------------------------------------------------------
__global__ void mma_prep_kernel(const float* __restrict__ wk, const float* __restrict__ wv,
                                uint32_t* __restrict__ frag, int heads)
{
    const int h = blockIdx.x;
    for (int w = threadIdx.x; w < kFragWordsPerHead; w += blockDim.x) {
        const bool value_side = w >= 2304;
        const int u = value_side ? w - 2304 : w;
        const int i = u & 3, lane = (u >> 2) & 31, mid = (u >> 7) & 1, t = u >> 8;
        const int g = lane >> 2, tig = lane & 3, r = i & 1;
        float lo, hi;
        if (!value_side) {
            const int nt = i >> 1, ks = mid;
            const int c0 = h * kHeadDim + 8 * tig + 4 * ks + 2 * r;
            if (nt == 0 || g == 0) {
                const int s = nt == 0 ? g : 8;
                const float e = (s == t) ? 1.f : 0.f;
                lo = wk[((size_t)c0 * 9 + s) * 9 + t] - e;
                hi = wk[((size_t)(c0 + 1) * 9 + s) * 9 + t] - e;
            } else {
                const int tap = g == 1 ? 0 : g;      // which tap's one-hot term this column sums
                lo = hi = (t == tap) ? 1.f : 0.f;
            }
        } else {
            const int j = 2 * mid + (i >> 1);
            const int c = h * kHeadDim + 8 * (g >> 1) + 2 * j + (g & 1);
            const int s0 = 2 * tig + 8 * r, s1 = s0 + 1;
            lo = s0 < 9 ? wv[((size_t)c * 9 + s0) * 9 + t] - (s0 == t ? 1.f : 0.f) : 0.f;
            hi = s1 < 9 ? wv[((size_t)c * 9 + s1) * 9 + t] - (s1 == t ? 1.f : 0.f) : 0.f;
        }
        frag[(size_t)h * kFragWordsPerHead + w] = pack_bf16(lo, hi);
    }
}

struct MmaParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    const uint32_t* frag;      // [heads][kFragWordsPerHead]
    const float* bias;         // [heads][9] or nullptr
    int* status;
    int B, H, W, heads;
    int TH, TW;                // tile size in pixels: TH % 4 == 0, TW % 8 == 0
    int tiles_x, tiles_y;
    float scale_log2e;         // log2(e) / sqrt(head_dim)
};

// ---------------------------------------------------------------------------------------------
// Main kernel.  grid = (tiles_x * tiles_y * B, heads), block = kWarps * 32.
// Dynamic shared memory: K halo | V halo | weight fragments | mbarrier.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kWarps * 32, 2)
mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
           const MmaParams P)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int HW2 = P.TW + 2;                               // halo row length in pixels
    const uint32_t halo_bytes = (uint32_t)(P.TH + 2) * HW2 * 64u;
    const uint32_t halo_pad = (halo_bytes + 127u) & ~127u;
    const unsigned char* sK = smem;                         // K halo  [TH+2][TW+2][32] bf16
    const unsigned char* sV = smem + halo_pad;              // V halo
    const unsigned char* sW = smem + 2 * halo_pad;          // weight fragments of this head
    const uint32_t bar = smem_u32(sW) + kFragWordsPerHead * 4;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int h = blockIdx.y;
    int tile = blockIdx.x;
    const int tx = tile % P.tiles_x; tile /= P.tiles_x;
    const int ty = tile % P.tiles_y;
    const int b = tile / P.tiles_y;
    const int x_org = tx * P.TW, y_org = ty * P.TH;        // tile origin in the map

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_expect_tx(bar, 2 * halo_bytes);
        tma_load_4d(smem_u32(sK), &map_k, bar, h * kHeadDim, x_org - 1, y_org - 1, b);
        tma_load_4d(smem_u32(sV), &map_v, bar, h * kHeadDim, x_org - 1, y_org - 1, b);
    }
    // weight fragments of this head -> shared memory (overlaps the TMA loads)
    {
        const uint4* src = reinterpret_cast<const uint4*>(P.frag + (size_t)h * kFragWordsPerHead);
        uint4* dst = reinterpret_cast<uint4*>(smem + 2 * halo_pad);
        for (int i = threadIdx.x; i < kFragWordsPerHead / 4; i += kWarps * 32) dst[i] = src[i];
    }
    // per-lane bias terms (slots 2*tig, 2*tig+1, and 8 on tig 0), in log2 units
    float bias0 = 0.f, bias1 = 0.f, bias8 = 0.f;
    if (P.bias) {
        const float* bh = P.bias + h * 9;
        bias0 = bh[2 * tig] * 1.4426950408889634f;
        bias1 = bh[2 * tig + 1] * 1.4426950408889634f;
        bias8 = bh[8] * 1.4426950408889634f;
    }
    __syncthreads();
    if (!mbar_wait(bar, 0)) {
        if (lane == 0) atomicExch(P.status, 1);
        return;
    }

    const int units_x = P.TW >> 3, units = units_x * (P.TH >> 2);
    const int C = P.heads * kHeadDim;
    const uint32_t ones_t1 = g == 0 ? kOnes : 0u;           // third n-tile: column 0 sums tap 1,
    const uint32_t ones_t8 = g == 1 ? kOnes : 0u;           //               column 1 sums tap 8

    for (int unit = warp; unit < units; unit += kWarps) {
        const int ux = (unit % units_x) * 8, uy = (unit / units_x) * 4;   // unit origin in the tile
        const int x = x_org + ux + g;                                     // this lane's column
        const int y0 = y_org + uy;
        if (y0 >= P.H || x_org + ux >= P.W) continue;                     // unit outside the map
        const bool x_in = x < P.W;

        // ---- q of the lane's four pixels, 8 channels each, straight from global memory ----
        uint32_t qf[4][4];
#pragma unroll
        for (int py = 0; py < 4; ++py) {
            uint4 v = make_uint4(0, 0, 0, 0);
            if (x_in && y0 + py < P.H)
                v = *reinterpret_cast<const uint4*>(P.q + ((size_t)(b * P.H + y0 + py) * P.W + x) * C + h * kHeadDim + tig * 8);
            qf[py][0] = v.x; qf[py][1] = v.y; qf[py][2] = v.z; qf[py][3] = v.w;
        }

        // halo address of (row uy + vy, column ux + g + dx): vy, dx count from the halo origin
        const uint32_t lane_off = ((uint32_t)(uy * HW2 + ux + g) * 64u) + tig * 16u;

        // ================= key side: logits =================
        float acc[2][3][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 3; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;

#pragma unroll
        for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                const int t = dy * 3 + dx;
                uint4 bk[2];
                bk[0] = lds128(sW, ((t * 2 + 0) * 32 + lane) * 16);
                bk[1] = lds128(sW, ((t * 2 + 1) * 32 + lane) * 16);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    // rows g / g+8 of MMA tile mt are pixel rows 2mt / 2mt+1; tap row = py + dy
                    const uint4 k0 = lds128(sK, lane_off + (uint32_t)((2 * mt + dy) * HW2 + dx) * 64u);
                    const uint4 k1 = lds128(sK, lane_off + (uint32_t)((2 * mt + 1 + dy) * HW2 + dx) * 64u);
                    uint32_t a0[4], a1[4];
                    a0[0] = hmul2_bf16(qf[2 * mt][0], k0.x);     a0[1] = hmul2_bf16(qf[2 * mt + 1][0], k1.x);
                    a0[2] = hmul2_bf16(qf[2 * mt][1], k0.y);     a0[3] = hmul2_bf16(qf[2 * mt + 1][1], k1.y);
                    a1[0] = hmul2_bf16(qf[2 * mt][2], k0.z);     a1[1] = hmul2_bf16(qf[2 * mt + 1][2], k1.z);
                    a1[2] = hmul2_bf16(qf[2 * mt][3], k0.w);     a1[3] = hmul2_bf16(qf[2 * mt + 1][3], k1.w);
                    mma_bf16(acc[mt][0], a0, bk[0].x, bk[0].y);
                    mma_bf16(acc[mt][1], a0, bk[0].z, bk[0].w);
                    mma_bf16(acc[mt][0], a1, bk[1].x, bk[1].y);
                    mma_bf16(acc[mt][1], a1, bk[1].z, bk[1].w);
                    if (t == 1) { mma_bf16(acc[mt][2], a0, ones_t1, ones_t1); mma_bf16(acc[mt][2], a1, ones_t1, ones_t1); }
                    if (t == 8) { mma_bf16(acc[mt][2], a0, ones_t8, ones_t8); mma_bf16(acc[mt][2], a1, ones_t8, ones_t8); }
                }
            }
        }

        // ================= softmax over the 9 slots (4 lanes of a quad share a pixel) =========
        // e0/e1: slots 2*tig, 2*tig+1; e8: slot 8 (tig 0 only, 0 elsewhere); unnormalised.
        float e0[4], e1[4], e8[4], inv[4];
#pragma unroll
        for (int py = 0; py < 4; ++py) {
            const int mt = py >> 1, o = (py & 1) * 2;
            const float x0 = acc[mt][0][o], x1 = acc[mt][0][o + 1];
            const float y0_ = acc[mt][1][o], y1_ = acc[mt][1][o + 1];
            const float z0 = acc[mt][2][o], z1 = acc[mt][2][o + 1];
            float l0, l1, l8;
            if (tig == 0) { l0 = x0 + y1_; l1 = x1 + z0; l8 = (y0_ + z1) * P.scale_log2e + bias8; }
            else          { l0 = x0 + y0_; l1 = x1 + y1_; l8 = -INFINITY; }
            l0 = l0 * P.scale_log2e + bias0;
            l1 = l1 * P.scale_log2e + bias1;
            float m = fmaxf(fmaxf(l0, l1), l8);
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            e0[py] = fast_exp2(l0 - m);
            e1[py] = fast_exp2(l1 - m);
            e8[py] = fast_exp2(l8 - m);           // exp2(-inf) = 0 on lanes without slot 8
            float s = e0[py] + e1[py] + e8[py];
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            inv[py] = 1.f / s;
        }

        // ================= value side =================
        float o_acc[4][8];
#pragma unroll
        for (int py = 0; py < 4; ++py)
#pragma unroll
            for (int i = 0; i < 8; ++i) o_acc[py][i] = 0.f;

        uint32_t af[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            af[mt][0] = pack_bf16(e0[2 * mt], e1[2 * mt]);
            af[mt][1] = pack_bf16(e0[2 * mt + 1], e1[2 * mt + 1]);
            af[mt][2] = pack_bf16(e8[2 * mt], 0.f);
            af[mt][3] = pack_bf16(e8[2 * mt + 1], 0.f);
        }
        const int quad = lane & ~3;

#pragma unroll
        for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                const int t = dy * 3 + dx;
                uint4 bv[2];
                bv[0] = lds128(sW, 9216 + ((t * 2 + 0) * 32 + lane) * 16);
                bv[1] = lds128(sW, 9216 + ((t * 2 + 1) * 32 + lane) * 16);
                const int src = quad | (t < 8 ? (t >> 1) : 0);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    // e[p, t] of both pixel rows, from the lane of the quad that owns slot t
                    const float ea = __shfl_sync(0xffffffffu, t == 8 ? e8[2 * mt] : ((t & 1) ? e1[2 * mt] : e0[2 * mt]), src);
                    const float eb = __shfl_sync(0xffffffffu, t == 8 ? e8[2 * mt + 1] : ((t & 1) ? e1[2 * mt + 1] : e0[2 * mt + 1]), src);
                    const uint4 v0 = lds128(sV, lane_off + (uint32_t)((2 * mt + dy) * HW2 + dx) * 64u);
                    const uint4 v1 = lds128(sV, lane_off + (uint32_t)((2 * mt + 1 + dy) * HW2 + dx) * 64u);
                    const uint32_t v0r[4] = {v0.x, v0.y, v0.z, v0.w};
                    const uint32_t v1r[4] = {v1.x, v1.y, v1.z, v1.w};
                    const uint32_t bvr[8] = {bv[0].x, bv[0].y, bv[0].z, bv[0].w, bv[1].x, bv[1].y, bv[1].z, bv[1].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float c[4] = {ea, ea, eb, eb};
                        mma_bf16(c, af[mt], bvr[2 * j], bvr[2 * j + 1]);
                        o_acc[2 * mt][2 * j]         = fmaf(c[0], bf16_lo(v0r[j]), o_acc[2 * mt][2 * j]);
                        o_acc[2 * mt][2 * j + 1]     = fmaf(c[1], bf16_hi(v0r[j]), o_acc[2 * mt][2 * j + 1]);
                        o_acc[2 * mt + 1][2 * j]     = fmaf(c[2], bf16_lo(v1r[j]), o_acc[2 * mt + 1][2 * j]);
                        o_acc[2 * mt + 1][2 * j + 1] = fmaf(c[3], bf16_hi(v1r[j]), o_acc[2 * mt + 1][2 * j + 1]);
                    }
                }
            }
        }

        // ================= normalise, convert, store (16 bytes per lane and pixel) =============
#pragma unroll
        for (int py = 0; py < 4; ++py) {
            if (x_in && y0 + py < P.H) {
                uint4 r;
                r.x = pack_bf16(o_acc[py][0] * inv[py], o_acc[py][1] * inv[py]);
                r.y = pack_bf16(o_acc[py][2] * inv[py], o_acc[py][3] * inv[py]);
                r.z = pack_bf16(o_acc[py][4] * inv[py], o_acc[py][5] * inv[py]);
                r.w = pack_bf16(o_acc[py][6] * inv[py], o_acc[py][7] * inv[py]);
                *reinterpret_cast<uint4*>(P.out + ((size_t)(b * P.H + y0 + py) * P.W + x) * C + h * kHeadDim + tig * 8) = r;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// [B][H][W][C] bf16 viewed as a 4-D tensor (C, W, H, B); box = 32 channels x (TW+2) x (TH+2) x 1.
bool make_halo_map(CUtensorMap* map, const void* base, int B, int H, int W, int C, int TH, int TW) {
    return make_tile_map(map, base, 2, B, H, W, C, kHeadDim, TW + 2, TH + 2);
}

void pick_tile(int H, int W, int* TH, int* TW, int* tiles_x, int* tiles_y) {
    const int tx = (W + 63) / 64;
    *TW = ((((W + tx - 1) / tx) + 7) / 8) * 8;
    *tiles_x = (W + *TW - 1) / *TW;
    *TH = H <= 4 ? 4 : 8;
    *tiles_y = (H + *TH - 1) / *TH;
}

size_t main_smem_bytes(int TH, int TW) {
    const size_t halo = (((size_t)(TH + 2) * (TW + 2) * 64) + 127) & ~(size_t)127;
    return 2 * halo + kFragWordsPerHead * 4 + 16;
}

}  // namespace

bool mma_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && ksize == 3;
}

size_t mma_workspace_bytes(int heads) { return (size_t)heads * kFragWordsPerHead * 4; }

// Per device, once: allow the main kernel its dynamic shared memory and resolve the driver
// entry point used to encode tensor maps.
cudaError_t mma_setup() {
    if (!tensor_map_available()) return cudaErrorNotSupported;
    return cudaFuncSetAttribute(mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t launch_mma_prep(const Problem& p, void* workspace, cudaStream_t stream) {
    mma_prep_kernel<<<p.heads, 256, 0, stream>>>(p.wk, p.wv, static_cast<uint32_t*>(workspace), p.heads);
    return cudaGetLastError();
}

cudaError_t launch_mma_main(const Problem& p, const void* workspace, int* d_status, cudaStream_t stream) {
    int TH, TW, tiles_x, tiles_y;
    pick_tile(p.H, p.W, &TH, &TW, &tiles_x, &tiles_y);
    const int C = p.heads * kHeadDim;
    CUtensorMap map_k, map_v;
    if (!make_halo_map(&map_k, p.k, p.B, p.H, p.W, C, TH, TW) ||
        !make_halo_map(&map_v, p.v, p.B, p.H, p.W, C, TH, TW))
        return cudaErrorInvalidValue;

    MmaParams P;
    P.q = static_cast<const __nv_bfloat16*>(p.q);
    P.out = static_cast<__nv_bfloat16*>(p.out);
    P.frag = static_cast<const uint32_t*>(workspace);
    P.bias = p.bias;
    P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.TH = TH; P.TW = TW; P.tiles_x = tiles_x; P.tiles_y = tiles_y;
    P.scale_log2e = 1.4426950408889634f / sqrtf((float)kHeadDim);

    const size_t smem = main_smem_bytes(TH, TW);
    const long long tiles = (long long)tiles_x * tiles_y * p.B;
    if (tiles > 0x7fffffffLL || p.heads > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)tiles, (unsigned)p.heads);
    mma_kernel<<<grid, kWarps * 32, smem, stream>>>(map_k, map_v, P);
    return cudaGetLastError();
}

}  // namespace slide_attn

// ---------------------------------------------------------------------------------------------
// Allocation-free entry point.
//
// Some callers may not allocate device memory at all: code running inside a memory-planned
// region (a framework's static arena, a plugin that is handed fixed buffers), a process whose
// allocator is locked down after start-up, or a latency-critical loop where cudaMalloc's implicit
// device synchronisation is not acceptable.  slide_attn_create allocates, so those callers cannot
// hold a context.  For them the scratch of the MMA variant (the re-laid-out weights and the
// status word) lives in the fixed arrays below, which every GPU that loads this library keeps
// until the process exits: kStaticMaxHeads * 18 432 B + 256 B = 288.25 KiB.
// ---------------------------------------------------------------------------------------------
namespace slide_attn {
namespace {

constexpr int kStaticMaxHeads = 16;
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) uint32_t g_static_frag[kStaticMaxHeads * kFragWordsPerHead];
static __device__ __align__(256) int g_static_status[64];

// In host code the two names above are host-side stand-ins, not device addresses; the addresses
// the kernels get are resolved per device with cudaGetSymbolAddress.
struct StaticScratch {
    bool ready;
    uint32_t* frag;
    int* status;
};
StaticScratch g_scratch[kStaticMaxDevices];
std::mutex g_scratch_mutex;

slide_attn_status static_scratch(int dev, StaticScratch* out) {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    StaticScratch& s = g_scratch[dev];
    if (!s.ready) {
        if (mma_setup() != cudaSuccess) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
        void* frag = nullptr;
        void* status = nullptr;
        if (cudaGetSymbolAddress(&frag, g_static_frag) != cudaSuccess ||
            cudaGetSymbolAddress(&status, g_static_status) != cudaSuccess || !frag || !status) {
            cudaGetLastError();
            return SLIDE_ATTN_ERR_CUDA;
        }
        s.frag = static_cast<uint32_t*>(frag);
        s.status = static_cast<int*>(status);
        s.ready = true;
    }
    *out = s;
    return SLIDE_ATTN_OK;
}

}  // namespace
}  // namespace slide_attn

extern "C" slide_attn_status slide_attn_forward_noalloc(
    const void* q, const void* k, const void* v, const float* wk, const float* wv, const float* bias,
    void* out, int B, int H, int W, int heads, int head_dim, int ksize, slide_attn_dtype dtype,
    void* cuda_stream)
{
    using namespace slide_attn;
    if (!q || !k || !v || !wk || !wv || !out) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (B < 1 || H < 1 || W < 1 || heads < 1 || head_dim < 1 || ksize < 1) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (dtype != SLIDE_ATTN_F32 && dtype != SLIDE_ATTN_BF16) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (out == q || out == k || out == v) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!mma_supports(dtype, head_dim, ksize)) return SLIDE_ATTN_ERR_UNSUPPORTED;
    if (heads > kStaticMaxHeads) return SLIDE_ATTN_ERR_TOO_LARGE;
    if ((long long)B * H * W > (1LL << 40) / ((long long)heads * head_dim)) return SLIDE_ATTN_ERR_TOO_LARGE;
    auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out) || misaligned(wk) ||
        misaligned(wv) || (bias && misaligned(bias)))
        return SLIDE_ATTN_ERR_ALIGNMENT;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    if (dev < 0 || dev >= kStaticMaxDevices) return SLIDE_ATTN_ERR_UNSUPPORTED;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    if (major != 10) return SLIDE_ATTN_ERR_ARCH;

    StaticScratch scratch;
    slide_attn_status st = static_scratch(dev, &scratch);
    if (st != SLIDE_ATTN_OK) return st;

    Problem p;
    p.B = B; p.H = H; p.W = W; p.heads = heads; p.head_dim = head_dim; p.ksize = ksize;
    p.has_bias = bias != nullptr; p.dtype = dtype;
    p.q = q; p.k = k; p.v = v; p.wk = wk; p.wv = wv; p.bias = bias; p.out = out;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The fragment words of the heads in use are all rewritten by the prep launch; the status
    // word is the only thing that has to start at zero.
    if (cudaMemsetAsync(scratch.status, 0, sizeof(int), stream) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    cudaError_t err = launch_mma_prep(p, scratch.frag, stream);
    if (err == cudaSuccess) err = launch_mma_main(p, scratch.frag, scratch.status, stream);
    return err == cudaSuccess ? SLIDE_ATTN_OK : SLIDE_ATTN_ERR_CUDA;
}
