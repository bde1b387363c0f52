// Shared by the staged CUDA-core kernels (fixed-shift fast path and the generic tile kernel): the tile
// geometry, the shared-memory plan of a halo tile in 64-byte channel planes, and the per-lane piece of
// eight channels.
//
// One CTA = one head of a 4 x 32 pixel tile (four warps; several CTAs share an SM, so one CTA's loads
// overlap another's arithmetic).  The K and V tile + floor(k/2) halo and the q tile come in by TMA
// (out-of-map elements zero-filled: that IS the padding of Fig. 2) as "planes" of 64 bytes of channels
// per pixel (bf16: one plane of 32 channels; fp32: two planes of 16), so that a quad of lanes reads one
// pixel's plane as four 16-byte pieces and a warp-wide load covers 512 contiguous bytes.  A warp owns 8
// columns x 4 rows; lane (g, tig) = column g, channels of piece tig: bf16 channels 8 tig .. 8 tig + 7,
// fp32 channels 4 tig .. 4 tig + 3 and 16 + 4 tig .. 16 + 4 tig + 3.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {
namespace tile {

constexpr int kHeadDim = 32;
constexpr int kTW = 32;                        // tile width in pixels
constexpr int kR = 4;                          // pixel rows per warp
constexpr float kLog2e = 1.4426950408889634f;

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> { static constexpr int planes = 1, th = 4; };
template <> struct Elem<float> { static constexpr int planes = 2, th = 4; };

template <typename T, int K>
struct Cfg {
    static constexpr int planes = Elem<T>::planes;
    static constexpr int TH = Elem<T>::th;
    static constexpr int warps = (kTW / 8) * (TH / kR);
    static constexpr int threads = warps * 32;
    static constexpr int HW = kTW + K - 1, HH = TH + K - 1;                 // halo tile
    static constexpr uint32_t halo_plane = (uint32_t)(HW * HH * 64 + 127) & ~127u;
    static constexpr uint32_t q_plane = (uint32_t)(kTW * TH * 64);
    static constexpr uint32_t k_off = 0, v_off = planes * halo_plane, q_off = 2 * planes * halo_plane;
    static constexpr uint32_t bias_off = q_off + planes * q_plane;
    static constexpr uint32_t bar_off = bias_off + ((K * K * 4 + 15) & ~15);
    static constexpr uint32_t total = bar_off + 16 + 128;                   // + alignment slack
    static constexpr uint32_t tx_bytes = planes * (2u * HW * HH * 64u + q_plane);
};

struct TileParams {
    const float* wt;                 // generic kernel: transposed weights wk^T then wv^T, [slot][tap][C]
    const float* bias;
    void* out;
    int* status;
    int B, H, W, heads;
    int tiles_x, tiles_y;
    float scale_log2e;
};

// Eight channels of one pixel (the piece of lane tig), as loaded and as floats.  bf16: one 16-byte load,
// kept packed for the q.k products (bf16 x bf16 + fp32 in one instruction, exact products) and widened
// for the value side; fp32: one 16-byte load per plane.
template <typename T> struct Piece;
template <> struct Piece<__nv_bfloat16> {
    struct Raw { uint32_t w[4]; };
    static __device__ __forceinline__ Raw load(const unsigned char* tile, uint32_t plane_bytes, uint32_t pix, int tig) {
        const uint4 v = *reinterpret_cast<const uint4*>(tile + pix * 64u + tig * 16u);
        Raw r; r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
        return r;
    }
    static __device__ __forceinline__ float dot(const Raw& a, const Raw& b) {
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            asm("{\n\t.reg .b16 al, ah, bl, bh;\n\t"
                "mov.b32 {al, ah}, %1;\n\tmov.b32 {bl, bh}, %2;\n\t"
                "fma.rn.f32.bf16 %0, al, bl, %0;\n\t"
                "fma.rn.f32.bf16 %0, ah, bh, %0;\n\t}"
                : "+f"(acc) : "r"(a.w[i]), "r"(b.w[i]));
        return acc;
    }
    static __device__ __forceinline__ void widen(const Raw& r, float (&f)[8]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[2 * i] = bf16_lo(r.w[i]); f[2 * i + 1] = bf16_hi(r.w[i]); }
    }
};
template <> struct Piece<float> {
    struct Raw { float f[8]; };
    static __device__ __forceinline__ Raw load(const unsigned char* tile, uint32_t plane_bytes, uint32_t pix, int tig) {
        const float4 a = *reinterpret_cast<const float4*>(tile + pix * 64u + tig * 16u);
        const float4 b = *reinterpret_cast<const float4*>(tile + plane_bytes + pix * 64u + tig * 16u);
        Raw r;
        r.f[0] = a.x; r.f[1] = a.y; r.f[2] = a.z; r.f[3] = a.w; r.f[4] = b.x; r.f[5] = b.y; r.f[6] = b.z; r.f[7] = b.w;
        return r;
    }
    static __device__ __forceinline__ float dot(const Raw& a, const Raw& b) {
        float p0 = a.f[0] * b.f[0], p1 = a.f[1] * b.f[1];
        ffma2(p0, p1, a.f[2], a.f[3], b.f[2], b.f[3]);
        ffma2(p0, p1, a.f[4], a.f[5], b.f[4], b.f[5]);
        ffma2(p0, p1, a.f[6], a.f[7], b.f[6], b.f[7]);
        return p0 + p1;
    }
    static __device__ __forceinline__ void widen(const Raw& r, float (&f)[8]) {
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = r.f[i];
    }
};

__device__ __forceinline__ void fmul2(float& a0, float& a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb;\n\t"
        "mov.b64 ra, {%0, %1};\n\tmov.b64 rb, {%2, %3};\n\t"
        "mul.rn.f32x2 ra, ra, rb;\n\t"
        "mov.b64 {%0, %1}, ra;\n\t}"
        : "+f"(a0), "+f"(a1) : "f"(b0), "f"(b1));
}


}  // namespace tile
}  // namespace slide_attn
