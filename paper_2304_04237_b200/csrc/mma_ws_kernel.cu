// MMA_WS variant (bf16, head_dim 32, k = 3): persistent, warp-specialised form of the tensor-core
// kernel.  Same arithmetic as mma_kernel.cu (w = E + D split, key-side contraction over
// (tap, channel), value-side contraction over slots with the exact fp32 e[p,t] as accumulator
// start; Eq. 2 with Eq. 12 inside), different schedule:
//
//   * one CTA per SM, each bound to ONE head for its whole life, looping over 4 x TW pixel tiles;
//   * key warps and value warps.  A key warp keeps all key-side B fragments (72 registers) and
//     turns a unit (4 rows x 8 columns) into unnormalised softmax weights e[p, 0..8] and 1/sum; a
//     value warp keeps all value-side B fragments and turns e into the output.  e travels through
//     small rings of shared-memory mailboxes (one ring per key/value warp pair), guarded by
//     mbarriers;
//   * K / V halo tiles and the q tile arrive by TMA (zero fill outside the map = the padding of the
//     convolution) into a 3-stage ring; lane 0 of key warp 0 is the producer;
//   * the fp32 weights of the head are brought in once by two 1-D bulk copies and every warp builds
//     its own fragments from them, so there is no separate weight-prep launch and no workspace.
//
// Lane (g, tig) = (lane/4, lane%4) owns column g of the unit, all four rows, and channels
// 8*tig .. 8*tig+7.  Pixel rows 2*mt and 2*mt+1 are rows g and g+8 of MMA tile mt, so the two halves
// of an MMA read the same halo column, one row apart.  The loops walk a halo column top to bottom:
// each halo position is loaded (and, on the value side, widened to fp32) once per lane and reused
// by every tap that touches it.  Lanes g and g+1 read adjacent 64-byte pixels, so every 16-byte
// shared-memory access is conflict-free without swizzling.
//
// Every wait is bounded; a wait that runs out sets the status word and the warp leaves.
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

namespace {

// Tuning knobs (compile time).
#ifndef SA_WS_KWARPS
#define SA_WS_KWARPS 6
#endif
#ifndef SA_WS_VWARPS
#define SA_WS_VWARPS 6
#endif

constexpr int kHeadDim = 32;
constexpr int kKWarps = SA_WS_KWARPS;
constexpr int kVWarps = SA_WS_VWARPS;
constexpr int kThreads = (kKWarps + kVWarps) * 32;
constexpr int kMaxStages = 3;
// Mailbox rings: unit u uses ring u % kRings, so every ring has exactly one writing key warp and
// one reading value warp, both walking it in order; kRingDepth slots per ring.
constexpr int kRings = kKWarps > kVWarps ? kKWarps : kVWarps;
constexpr int kRingDepth = 2;
constexpr int kMailSlots = kRings * kRingDepth;
static_assert(kRings % kKWarps == 0 && kRings % kVWarps == 0, "one warp count must divide the other");
static_assert(kMailSlots <= 16, "barrier table holds 16 mailbox slots");
constexpr int kMailBytes = 8 * 10 * 4 * 4;              // [g 8][slot 0..8, 9 = 1/sum][pixel 4] floats
constexpr int kWeightBytes = kHeadDim * 81 * 4;         // fp32 weights of one head, one side
constexpr float kLog2e = 1.4426950408889634f;

struct WsParams {
    const float* wk;
    const float* wv;
    const float* bias;         // [heads][9] or nullptr
    __nv_bfloat16* out;
    int* status;
    int B, H, W, heads;
    int TW;                    // tile width in pixels (multiple of 8); tile height is 4
    int tiles_x, tiles_y;
    int stages;                // 2 or 3
    float scale_log2e;         // log2(e) / sqrt(head_dim)
};

struct Smem {
    uint32_t halo_pad;         // bytes of one K or V halo tile (6 rows x (TW+2) pixels x 64 B), 1024-aligned
    uint32_t stage_bytes;      // K halo | V halo | q tile, 1024-aligned
    uint32_t mail_off;         // mailboxes: [kMailSlots][kMailBytes]
    uint32_t bar_off;          // mbarriers
    uint32_t total;            // including 1024 bytes of slack to align the base
};

__host__ __device__ inline Smem smem_layout(int TW, int stages) {
    Smem s;
    s.halo_pad = ((uint32_t)(6 * (TW + 2) * 64) + 1023u) & ~1023u;
    s.stage_bytes = 2 * s.halo_pad + (((uint32_t)(4 * TW * 64) + 1023u) & ~1023u);
    // the last stage doubles as the staging area of the head's fp32 weights (both sides)
    const uint32_t wbytes = ((uint32_t)(2 * kWeightBytes) + 1023u) & ~1023u;
    if (s.stage_bytes < wbytes) s.stage_bytes = wbytes;
    s.mail_off = s.stage_bytes * stages;
    s.bar_off = s.mail_off + kMailSlots * kMailBytes;
    s.total = s.bar_off + 64 * 8 + 1024;
    return s;
}

// barrier indices (8 bytes each) behind bar_off
constexpr int kBarFull = 0;        // [stage]  TMA landed
constexpr int kBarEmpty = 3;       // [stage]  all units of the tile are done with the stage
constexpr int kBarMailFull = 6;    // [slot]   e written
constexpr int kBarMailEmpty = 22;  // [slot]   e consumed
constexpr int kBarWeights = 38;    // weights landed
constexpr int kBarWeightsDone = 39;  // all warps have built their fragments

__device__ __forceinline__ float4 lds_f4(const unsigned char* base, uint32_t off) {
    return *reinterpret_cast<const float4*>(base + off);
}
__device__ __forceinline__ uint4 lds_u4(const unsigned char* base, uint32_t off) {
    return *reinterpret_cast<const uint4*>(base + off);
}

__global__ void __launch_bounds__(kThreads, 1)
mma_ws_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_v, const WsParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-aligned
    const Smem L = smem_layout(P.TW, P.stages);
    const uint32_t bar0 = smem_u32(smem + L.bar_off);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int S = P.stages;
    const int U = P.TW >> 3;                                   // units per tile
    const int HW2 = P.TW + 2;

    // this CTA's head and its share of that head's tiles
    const int h = blockIdx.x % P.heads;
    const int rank = blockIdx.x / P.heads;
    const int nrank = ((int)gridDim.x - h + P.heads - 1) / P.heads;
    const int tiles_per_head = P.B * P.tiles_y * P.tiles_x;
    const int my_tiles = rank < tiles_per_head ? (tiles_per_head - rank + nrank - 1) / nrank : 0;
    const int C = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar(kBarFull + s), 1);
            mbar_init(bar(kBarEmpty + s), kKWarps + kVWarps);
        }
        for (int i = 0; i < kMailSlots; ++i) {
            mbar_init(bar(kBarMailFull + i), 1);
            mbar_init(bar(kBarMailEmpty + i), 1);
        }
        mbar_init(bar(kBarWeights), 1);
        mbar_init(bar(kBarWeightsDone), kKWarps + kVWarps);
    }
    __syncthreads();
    if (my_tiles == 0) return;

    // tile n of this CTA -> stage n % S
    auto issue_tile = [&](int n) {
        const int gt = rank + n * nrank;
        const int tx = gt % P.tiles_x;
        const int ty = (gt / P.tiles_x) % P.tiles_y;
        const int b = gt / (P.tiles_x * P.tiles_y);
        const int s = n % S;
        const uint32_t base = smem_u32(smem + (size_t)s * L.stage_bytes);
        const uint32_t fb = bar(kBarFull + s);
        mbar_expect_tx(fb, (uint32_t)(2 * 6 * HW2 * 64 + 4 * P.TW * 64));
        tma_load_4d(base, &map_k, fb, h * kHeadDim, tx * P.TW - 1, ty * 4 - 1, b);
        tma_load_4d(base + L.halo_pad, &map_v, fb, h * kHeadDim, tx * P.TW - 1, ty * 4 - 1, b);
        tma_load_4d(base + 2 * L.halo_pad, &map_q, fb, h * kHeadDim, tx * P.TW, ty * 4, b);
    };

    // The fp32 weights of the head are staged in the LAST stage's memory; that stage receives its
    // first tile only after every warp has built its fragments.
    const unsigned char* w_stage = smem + (size_t)(S - 1) * L.stage_bytes;
    int issued = 0;                                            // producer state (key warp 0, lane 0)
    if (warp == 0 && lane == 0) {
        mbar_expect_tx(bar(kBarWeights), 2 * kWeightBytes);
        bulk_load_1d(smem_u32(w_stage), P.wk + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
        bulk_load_1d(smem_u32(w_stage) + kWeightBytes, P.wv + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
        while (issued < my_tiles && issued < S - 1) issue_tile(issued++);
    }
    __syncwarp();

    // Issues every tile whose stage is free.  A tile that key warp 0 itself needs now (index <=
    // `need`) is waited for; later ones are only probed.  Returns false if a wait ran out.
    auto produce = [&](int need) -> bool {
        while (issued < my_tiles) {
            uint32_t b = 0, par = 0;
            bool gated = false;
            if (issued == S - 1) { b = bar(kBarWeightsDone); par = 0; gated = true; }   // staging area must be dead
            else if (issued >= S) { b = bar(kBarEmpty + issued % S); par = ((issued / S) - 1) & 1; gated = true; }
            if (gated && !mbar_test(b, par)) {
                if (issued > need) return true;               // not needed yet: try again later
                if (!mbar_wait(b, par)) return false;
            }
            issue_tile(issued++);
        }
        return true;
    };

    bool ok = mbar_wait(bar(kBarWeights), 0);
    const float* wks = reinterpret_cast<const float*>(w_stage);
    const float* wvs = wks + kHeadDim * 81;

    if (warp < kKWarps) {
        // =====================================================================================
        // key warps
        // =====================================================================================
        uint32_t bk[9][2][4];          // [tap][k-step][n-tile 0: r0 r1 | n-tile 1: r0 r1]
        if (ok) {
#pragma unroll
            for (int t = 0; t < 9; ++t)
#pragma unroll
                for (int ks = 0; ks < 2; ++ks)
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const int c0 = 8 * tig + 4 * ks + 2 * r;
                        {   // n-tile 0: column g = slot g
                            const float e = (g == t) ? 1.f : 0.f;
                            bk[t][ks][r] = pack_bf16(wks[c0 * 81 + g * 9 + t] - e, wks[(c0 + 1) * 81 + g * 9 + t] - e);
                        }
                        {   // n-tile 1: column 0 = slot 8; column 1 sums tap 0; column n >= 2 sums tap n
                            const float e = (t == 8) ? 1.f : 0.f;
                            const uint32_t d = pack_bf16(wks[c0 * 81 + 72 + t] - e, wks[(c0 + 1) * 81 + 72 + t] - e);
                            const int tap = g == 1 ? 0 : g;
                            bk[t][ks][2 + r] = g == 0 ? d : (t == tap ? kOnesBf16x2 : 0u);
                        }
                    }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarWeightsDone));

        float bias0 = 0.f, bias1 = 0.f, bias8 = 0.f;
        if (P.bias) {
            const float* bh = P.bias + h * 9;
            bias0 = bh[2 * tig] * kLog2e;
            bias1 = bh[2 * tig + 1] * kLog2e;
            bias8 = bh[8] * kLog2e;
        }
        const uint32_t ones_t1 = g == 0 ? kOnesBf16x2 : 0u;    // third n-tile: column 0 sums tap 1,
        const uint32_t ones_t8 = g == 1 ? kOnesBf16x2 : 0u;    //               column 1 sums tap 8

        // Every warp visits every tile in order (waits for it, arrives on its release barrier), even
        // a tile in which it owns no unit: a warp that skipped a phase of a barrier could later
        // mistake an older phase for the one it waits for.
        for (int ti = 0; ok && ti < my_tiles; ++ti) {
            // ---- producer duty (key warp 0, lane 0): keep the ring filled -------------------
            if (warp == 0) {
                if (lane == 0 && !produce(ti)) ok = false;
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
            }
            const int stage = ti % S;
            if (!mbar_wait(bar(kBarFull + stage), (ti / S) & 1)) { ok = false; break; }
            const int u0 = ti * U;
          for (int ul = (warp + kKWarps - u0 % kKWarps) % kKWarps; ul < U; ul += kKWarps) {
            const int u = u0 + ul;
            const int ux = ul * 8;

            const unsigned char* sK = smem + (size_t)stage * L.stage_bytes;
            const unsigned char* sQ = sK + 2 * L.halo_pad;
            // q of the lane's four pixels (rows 0..3 of column ux + g)
            uint32_t qf[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = lds_u4(sQ, (uint32_t)(i * P.TW + ux + g) * 64u + tig * 16u);
                qf[i][0] = v.x; qf[i][1] = v.y; qf[i][2] = v.z; qf[i][3] = v.w;
            }
            // halo position (row r, column dx) of the lane's strip: pixel slot n0 + r*HW2 + dx
            const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;

            float acc[2][3][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < 3; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;

#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                uint4 kc[6];                                       // one halo column, rows 0..5
#pragma unroll
                for (int r = 0; r < 6; ++r) kc[r] = lds_u4(sK, off0 + (uint32_t)(r * HW2 + dx) * 64u);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                    for (int dy = 0; dy < 3; ++dy) {
                        const int t = dy * 3 + dx;
                        const uint4 k0 = kc[2 * mt + dy], k1 = kc[2 * mt + dy + 1];   // pixel rows 2mt / 2mt+1
                        uint32_t a0[4], a1[4];
                        a0[0] = hmul2_bf16(qf[2 * mt][0], k0.x);  a0[1] = hmul2_bf16(qf[2 * mt + 1][0], k1.x);
                        a0[2] = hmul2_bf16(qf[2 * mt][1], k0.y);  a0[3] = hmul2_bf16(qf[2 * mt + 1][1], k1.y);
                        a1[0] = hmul2_bf16(qf[2 * mt][2], k0.z);  a1[1] = hmul2_bf16(qf[2 * mt + 1][2], k1.z);
                        a1[2] = hmul2_bf16(qf[2 * mt][3], k0.w);  a1[3] = hmul2_bf16(qf[2 * mt + 1][3], k1.w);
                        mma_bf16(acc[mt][0], a0, bk[t][0][0], bk[t][0][1]);
                        mma_bf16(acc[mt][1], a0, bk[t][0][2], bk[t][0][3]);
                        mma_bf16(acc[mt][0], a1, bk[t][1][0], bk[t][1][1]);
                        mma_bf16(acc[mt][1], a1, bk[t][1][2], bk[t][1][3]);
                        if (t == 1) { mma_bf16(acc[mt][2], a0, ones_t1, ones_t1); mma_bf16(acc[mt][2], a1, ones_t1, ones_t1); }
                        if (t == 8) { mma_bf16(acc[mt][2], a0, ones_t8, ones_t8); mma_bf16(acc[mt][2], a1, ones_t8, ones_t8); }
                    }
                }
            }
            // softmax over the 9 slots; the 4 lanes of a quad share a pixel
            float e0[4], e1[4], e8[4], inv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int mt = i >> 1, o = (i & 1) * 2;
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
                e0[i] = fast_exp2(l0 - m);
                e1[i] = fast_exp2(l1 - m);
                e8[i] = fast_exp2(l8 - m);
                float s = e0[i] + e1[i] + e8[i];
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                s += __shfl_xor_sync(0xffffffffu, s, 2);
                inv[i] = 1.f / s;
            }

            const int seq = u / kRings;                                 // position in ring u % kRings
            const int slot = (u % kRings) * kRingDepth + seq % kRingDepth;
            if (!mbar_wait(bar(kBarMailEmpty + slot), ((seq / kRingDepth) & 1) ^ 1)) { ok = false; break; }
            unsigned char* mail = smem + L.mail_off + (size_t)slot * kMailBytes;
            *reinterpret_cast<float4*>(mail + (g * 10 + 2 * tig) * 16) = make_float4(e0[0], e0[1], e0[2], e0[3]);
            *reinterpret_cast<float4*>(mail + (g * 10 + 2 * tig + 1) * 16) = make_float4(e1[0], e1[1], e1[2], e1[3]);
            if (tig == 0) *reinterpret_cast<float4*>(mail + (g * 10 + 8) * 16) = make_float4(e8[0], e8[1], e8[2], e8[3]);
            if (tig == 1) *reinterpret_cast<float4*>(mail + (g * 10 + 9) * 16) = make_float4(inv[0], inv[1], inv[2], inv[3]);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarMailFull + slot));
          }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarEmpty + stage));  // this warp is done with the stage
        }
    } else {
        // =====================================================================================
        // value warps
        // =====================================================================================
        const int vw = warp - kKWarps;
        uint32_t bv[9][4][2];          // [tap][n-tile j][r]
        if (ok) {
#pragma unroll
            for (int t = 0; t < 9; ++t)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = 8 * (g >> 1) + 2 * j + (g & 1);
                    const int s0 = 2 * tig, s1 = 2 * tig + 1;
                    bv[t][j][0] = pack_bf16(wvs[c * 81 + s0 * 9 + t] - (s0 == t ? 1.f : 0.f),
                                            wvs[c * 81 + s1 * 9 + t] - (s1 == t ? 1.f : 0.f));
                    const uint32_t d8 = pack_bf16(wvs[c * 81 + 72 + t] - (t == 8 ? 1.f : 0.f), 0.f);
                    bv[t][j][1] = tig == 0 ? d8 : 0u;
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarWeightsDone));

        for (int ti = 0; ok && ti < my_tiles; ++ti) {
            const int gt = rank + ti * nrank;
            const int tx = gt % P.tiles_x;
            const int ty = (gt / P.tiles_x) % P.tiles_y;
            const int b = gt / (P.tiles_x * P.tiles_y);
            const int stage = ti % S;
            if (!mbar_wait(bar(kBarFull + stage), (ti / S) & 1)) { ok = false; break; }
            const int u0 = ti * U;
          for (int ul = (vw + kVWarps - u0 % kVWarps) % kVWarps; ul < U; ul += kVWarps) {
            const int u = u0 + ul;
            const int ux = ul * 8;
            const int seq = u / kRings;
            const int slot = (u % kRings) * kRingDepth + seq % kRingDepth;
            if (!mbar_wait(bar(kBarMailFull + slot), (seq / kRingDepth) & 1)) { ok = false; break; }
            const unsigned char* mail = smem + L.mail_off + (size_t)slot * kMailBytes;
            const unsigned char* sV = smem + (size_t)stage * L.stage_bytes + L.halo_pad;
            const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;

            uint32_t af[2][4];
            float4 invv;
            {
                const float4 lo = lds_f4(mail, (g * 10 + 2 * tig) * 16);
                const float4 hi = lds_f4(mail, (g * 10 + 2 * tig + 1) * 16);
                const float4 e8v = lds_f4(mail, (g * 10 + 8) * 16);
                invv = lds_f4(mail, (g * 10 + 9) * 16);
                af[0][0] = pack_bf16(lo.x, hi.x);  af[0][1] = pack_bf16(lo.y, hi.y);
                af[1][0] = pack_bf16(lo.z, hi.z);  af[1][1] = pack_bf16(lo.w, hi.w);
                af[0][2] = tig == 0 ? pack_bf16(e8v.x, 0.f) : 0u;  af[0][3] = tig == 0 ? pack_bf16(e8v.y, 0.f) : 0u;
                af[1][2] = tig == 0 ? pack_bf16(e8v.z, 0.f) : 0u;  af[1][3] = tig == 0 ? pack_bf16(e8v.w, 0.f) : 0u;
            }
            float o_acc[4][8];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int c = 0; c < 8; ++c) o_acc[i][c] = 0.f;

#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                // one halo column of the strip, rows 0..5, widened to fp32 once
                float vf[6][8];
#pragma unroll
                for (int r = 0; r < 6; ++r) {
                    const uint4 v = lds_u4(sV, off0 + (uint32_t)(r * HW2 + dx) * 64u);
                    vf[r][0] = bf16_lo(v.x); vf[r][1] = bf16_hi(v.x);
                    vf[r][2] = bf16_lo(v.y); vf[r][3] = bf16_hi(v.y);
                    vf[r][4] = bf16_lo(v.z); vf[r][5] = bf16_hi(v.z);
                    vf[r][6] = bf16_lo(v.w); vf[r][7] = bf16_hi(v.w);
                }
#pragma unroll
                for (int r = 0; r < 5; ++r) {                      // rows r (half 0) and r+1 (half 1)
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        const int dy = r - 2 * mt;
                        if (dy < 0 || dy > 2) continue;
                        const int t = dy * 3 + dx;
                        const float4 et = lds_f4(mail, (g * 10 + t) * 16);       // e[pixel 0..3][t]
                        const float ea = mt == 0 ? et.x : et.z, eb = mt == 0 ? et.y : et.w;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float d[4];
                            mma_bf16_c(d, af[mt], bv[t][j][0], bv[t][j][1], ea, ea, eb, eb);
                            ffma2(o_acc[2 * mt][2 * j], o_acc[2 * mt][2 * j + 1], d[0], d[1],
                                  vf[r][2 * j], vf[r][2 * j + 1]);
                            ffma2(o_acc[2 * mt + 1][2 * j], o_acc[2 * mt + 1][2 * j + 1], d[2], d[3],
                                  vf[r + 1][2 * j], vf[r + 1][2 * j + 1]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarMailEmpty + slot));

            const float invr[4] = {invv.x, invv.y, invv.z, invv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int y = ty * 4 + i, x = tx * P.TW + ux + g;
                if (y < P.H && x < P.W) {
                    uint4 r;
                    r.x = pack_bf16(o_acc[i][0] * invr[i], o_acc[i][1] * invr[i]);
                    r.y = pack_bf16(o_acc[i][2] * invr[i], o_acc[i][3] * invr[i]);
                    r.z = pack_bf16(o_acc[i][4] * invr[i], o_acc[i][5] * invr[i]);
                    r.w = pack_bf16(o_acc[i][6] * invr[i], o_acc[i][7] * invr[i]);
                    *reinterpret_cast<uint4*>(P.out + ((size_t)(b * P.H + y) * P.W + x) * C + h * kHeadDim + tig * 8) = r;
                }
            }
          }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarEmpty + stage));  // this warp is done with the stage
        }
    }
    if (!ok && lane == 0) atomicExch(P.status, 1);
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [B][H][W][C] bf16 as a 4-D tensor (C, W, H, B); box = 32 channels x bw pixels x bh rows x 1 image.
bool make_map(CUtensorMap* map, const void* base, int B, int H, int W, int C, int bw, int bh) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kHeadDim, (cuuint32_t)bw, (cuuint32_t)bh, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kMaxSmem = 227 * 1024;

}  // namespace

bool mma_ws_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && ksize == 3;
}

cudaError_t mma_ws_setup() {
    if (!encode_fn()) return cudaErrorNotSupported;
    return cudaFuncSetAttribute(mma_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

cudaError_t launch_mma_ws(const Problem& p, int* d_status, int num_sms, cudaStream_t stream) {
    // tile width: a multiple of 8 up to 64, splitting the row evenly
    const int txn = (p.W + 63) / 64;
    const int TW = ((((p.W + txn - 1) / txn) + 7) / 8) * 8;
    WsParams P;
    P.wk = p.wk; P.wv = p.wv; P.bias = p.bias;
    P.out = static_cast<__nv_bfloat16*>(p.out);
    P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.TW = TW;
    P.tiles_x = (p.W + TW - 1) / TW;
    P.tiles_y = (p.H + 3) / 4;
    P.stages = smem_layout(TW, 3).total <= kMaxSmem ? 3 : 2;
    P.scale_log2e = kLog2e / sqrtf((float)kHeadDim);
    const Smem L = smem_layout(TW, P.stages);
    if (L.total > kMaxSmem) return cudaErrorInvalidConfiguration;

    const int C = p.heads * kHeadDim;
    CUtensorMap map_q, map_k, map_v;
    if (!make_map(&map_q, p.q, p.B, p.H, p.W, C, TW, 4) ||
        !make_map(&map_k, p.k, p.B, p.H, p.W, C, TW + 2, 6) ||
        !make_map(&map_v, p.v, p.B, p.H, p.W, C, TW + 2, 6))
        return cudaErrorInvalidValue;

    const long long tiles = (long long)P.tiles_x * P.tiles_y * p.B * p.heads;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    int grid = num_sms;
    if (grid < p.heads) grid = p.heads;                    // every head needs at least one CTA
    if ((long long)grid > tiles) grid = (int)tiles;
    mma_ws_kernel<<<grid, kThreads, L.total, stream>>>(map_q, map_k, map_v, P);
    return cudaGetLastError();
}

}  // namespace slide_attn
