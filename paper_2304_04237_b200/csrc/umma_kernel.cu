// UMMA variant (bf16, head_dim 32, k = 3): like MMA_WS a persistent, warp-specialised kernel, but the
// value-side contraction runs on the 5th-generation tensor core (tcgen05.mma) with its accumulator
// in tensor memory.
//
// Arithmetic (Eq. 2 with Eq. 12 inside; w = E + D split as in mma_kernel.cu):
//   key side    logit[p,s] = sum_{t,c} q[p,c] k[p+off(t),c] (D_k[c,s,t] + [t == s])   mma.sync, key warps
//   softmax     e[p,s] = exp(logit - max)                                               key warps
//   value side  A'[p,(t,c)] = sum_s e[p,s] (D_v[c,s,t] + [t == s])                      tcgen05.mma
//               sum[p]      = sum_s e[p,s]                                              (16 extra columns)
//               out[p,c]    = (sum_t A'[p,t,c] v[p+off(t),c]) / sum[p]                  value warps
//
// The value-side product is one [128 pixels x 32] x [32 x 304] bf16 MMA per block of four units:
//   A row p (shared memory, written by the key warps):  e_hi[0..7] | e_hi[0..7] | e_lo[0..7] |
//                                                       e_hi[8], e_hi[8], e_lo[8], 0 ...
//     with e = e_hi + e_lo split into two bf16 values, so that the one-hot part is carried to
//     2^-17 relative accuracy while D_v only meets e_hi;
//   B column (t,c) (shared memory, built once per CTA):  D_v[c][0..7][t] | [s == t] | [s == t] |
//                                                       D_v[c][8][t], [t == 8], [t == 8], 0 ...
//   16 more columns hold 0 | 1 | 1 | 0,1,1,0... and so deliver sum_s e[p,s].
// D (fp32) lives in tensor memory, pixel = TMEM lane.  Columns are ordered by tap column dx; the
// three taps of one dx (96 columns; the last dx also carries the 16 sum columns) form a chunk.  The
// two sets of value warps (even / odd blocks) each own two 112-column TMEM slots and walk them as
// a ring, so while a set reads one chunk the MMA of its next chunk is already running.  Value warp w reads TMEM lanes 32w .. 32w+31 (its
// quadrant) with tcgen05.ld.16x256b, whose register layout equals the mma.sync accumulator fragment.
//
// Roles (16 warps, 128 registers each): warps 0-7 value warps (warp % 4 = TMEM quadrant = unit index
// within a block; warps w and w+4 take alternate blocks), warps 8-14 key warps (their B fragments
// are re-read from shared memory for every unit), warp 15 allocates / frees tensor memory and its
// lane 0 is the scheduler: it issues the TMA loads and the MMAs.  K (+ q) tiles and V tiles travel
// in separate TMA rings, so the key warps can run ahead of the value warps by as many blocks as
// there are A tiles.  Every wait is bounded; a wait that runs out sets
// the status word, and tensor memory is released on every path.
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

namespace {

constexpr int kHeadDim = 32;
constexpr int kVWarps = 8;
constexpr int kKWarps = 7;
constexpr int kCtlWarp = kVWarps + kKWarps;             // warp 15
constexpr int kThreads = (kVWarps + kKWarps + 1) * 32;
constexpr int kKStages = 2;                             // ring of K halo + q tiles
constexpr int kMaxVStages = 4;                          // ring of V halo tiles
constexpr int kABufs = 4;                               // A tiles (one per block in flight)
constexpr int kBkBytes = 9 * 2 * 32 * 16;               // key-side B fragments of the head, fragment order
constexpr int kABytes = 128 * 64;                       // 128 rows x 32 bf16
constexpr int kBCols = 304;                             // 288 value columns + 16 sum columns
constexpr int kBBytes = kBCols * 64;
constexpr int kWeightBytes = kHeadDim * 81 * 4;         // fp32 weights of one head, one side
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kTmemCols = 512;
constexpr int kDSlots = 4;                              // two TMEM chunk slots per value-warp set
constexpr uint32_t kDSlotCols = 112;
constexpr uint32_t kIdesc96 = umma_idesc_bf16(128, 96);
constexpr uint32_t kIdesc112 = umma_idesc_bf16(128, 112);

struct UmmaParams {
    const float* wk;
    const float* wv;
    const float* bias;         // [heads][9] or nullptr
    __nv_bfloat16* out;
    int* status;
    int B, H, W, heads;
    int TW;                    // tile width in pixels (multiple of 8); tile height is 4
    int tiles_x, tiles_y;
    int stages;                // depth of the V ring (2..4)
    float scale_log2e;         // log2(e) / sqrt(head_dim)
};

struct Smem {
    uint32_t halo_pad;         // bytes of one K or V halo tile (6 rows x (TW+2) pixels x 64 B), 1024-aligned
    uint32_t kstage_bytes;     // K halo | q tile
    uint32_t v_off;            // V ring [vstages][halo_pad]
    uint32_t b_off;            // B tile of the value-side MMA
    uint32_t bk_off;           // key-side B fragments [tap][k-step][lane][4 words]
    uint32_t a_off;            // A tiles [kABufs][kABytes]
    uint32_t tmem_off;         // TMEM base address written by tcgen05.alloc
    uint32_t bar_off;          // mbarriers
    uint32_t total;            // including 1024 bytes of slack to align the base
};

__host__ __device__ inline Smem smem_layout(int TW, int vstages) {
    Smem s;
    s.halo_pad = ((uint32_t)(6 * (TW + 2) * 64) + 1023u) & ~1023u;
    // a V stage doubles as the staging area of the head's fp32 weights (both sides)
    const uint32_t wbytes = ((uint32_t)(2 * kWeightBytes) + 1023u) & ~1023u;
    if (s.halo_pad < wbytes) s.halo_pad = wbytes;
    s.kstage_bytes = s.halo_pad + (((uint32_t)(4 * TW * 64) + 1023u) & ~1023u);
    s.v_off = kKStages * s.kstage_bytes;
    s.b_off = s.v_off + vstages * s.halo_pad;
    s.bk_off = s.b_off + kBBytes;
    s.a_off = s.bk_off + kBkBytes;
    s.tmem_off = s.a_off + kABufs * kABytes;
    s.bar_off = s.tmem_off + 16;
    s.total = s.bar_off + 32 * 8 + 1024;
    return s;
}

// barrier indices (8 bytes each) behind bar_off
constexpr int kBarKFull = 0;         // [K stage]  K halo and q tile landed
constexpr int kBarKEmpty = 2;        // [K stage]  every key warp is done with the stage
constexpr int kBarVFull = 4;         // [V stage]  V halo landed
constexpr int kBarVEmpty = 8;        // [V stage]  every value warp is done with the stage
constexpr int kBarWeights = 12;      // weights landed
constexpr int kBarWeightsDone = 13;  // all warps are done with the weight staging area
constexpr int kBarAReady = 14;       // [A buffer]  the 4 units of a block have written their rows
constexpr int kBarAFree = 18;        // [A buffer]  the MMAs reading the buffer are complete
constexpr int kBarDFull = 22;        // [TMEM slot]  MMA results of a chunk are in tensor memory
constexpr int kBarDFree = 26;        // [TMEM slot]  the 4 value warps of the set are done reading the chunk
constexpr int kBarVDone = 30;        // value warps have finished all TMEM reads

__device__ __forceinline__ uint4 lds_u4(const unsigned char* base, uint32_t off) {
    return *reinterpret_cast<const uint4*>(base + off);
}

// Bounded wait whose verdict is the same in all lanes of the (converged) warp.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}

__global__ void __launch_bounds__(kThreads, 1)
umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
            const __grid_constant__ CUtensorMap map_v, const UmmaParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-aligned
    const Smem L = smem_layout(P.TW, P.stages);
    const uint32_t bar0 = smem_u32(smem + L.bar_off);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    const int SV = P.stages;                                   // V ring depth
    const int U = P.TW >> 3;                                   // units per tile
    const int HW2 = P.TW + 2;

    // this CTA's head and its share of that head's tiles
    const int h = blockIdx.x % P.heads;
    const int rank = blockIdx.x / P.heads;
    const int nrank = ((int)gridDim.x - h + P.heads - 1) / P.heads;
    const int tiles_per_head = P.B * P.tiles_y * P.tiles_x;
    const int my_tiles = rank < tiles_per_head ? (tiles_per_head - rank + nrank - 1) / nrank : 0;
    const int my_units = my_tiles * U;
    const int my_blocks = (my_units + 3) >> 2;                 // blocks of four units = 128 pixels
    const int C = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kKStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKEmpty + s), kKWarps);
        }
        for (int s = 0; s < kMaxVStages; ++s) {
            mbar_init(bar(kBarVFull + s), 1);
            mbar_init(bar(kBarVEmpty + s), kVWarps);
        }
        mbar_init(bar(kBarWeights), 1);
        mbar_init(bar(kBarWeightsDone), kKWarps + kVWarps + 1);
        for (int i = 0; i < kABufs; ++i) {
            mbar_init(bar(kBarAReady + i), 4);
            mbar_init(bar(kBarAFree + i), 1);
        }
        for (int i = 0; i < kDSlots; ++i) {
            mbar_init(bar(kBarDFull + i), 1);
            mbar_init(bar(kBarDFree + i), 4);
        }
        mbar_init(bar(kBarVDone), kVWarps);
    }
    // A tiles start as zeros: the columns no key warp ever writes must not hold NaN patterns
    for (int i = threadIdx.x; i < kABufs * kABytes / 16; i += kThreads)
        reinterpret_cast<uint4*>(smem + L.a_off)[i] = make_uint4(0, 0, 0, 0);
    if (warp == kCtlWarp) tmem_alloc(smem_u32(smem + L.tmem_off), kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<const volatile uint32_t*>(smem + L.tmem_off);

    // Tile n of this CTA is global tile rank + n * nrank -> K stage n % kKStages, V stage n % SV.
    // Whoever walks the tiles keeps (tx, ty, b) and a stage counter and steps them without dividing:
    // a division costs a lone thread some hundred cycles, and the control thread has none to spare.
    struct TileWalk { int tx, ty, b, stage, round; };
    const int step_tx = nrank % P.tiles_x, step_ty = (nrank / P.tiles_x) % P.tiles_y,
              step_b = nrank / (P.tiles_x * P.tiles_y);
    auto walk_begin = [&]() {
        TileWalk w;
        w.tx = rank % P.tiles_x;
        w.ty = (rank / P.tiles_x) % P.tiles_y;
        w.b = rank / (P.tiles_x * P.tiles_y);
        w.stage = 0; w.round = 0;
        return w;
    };
    auto walk_next = [&](TileWalk& w, int nstages) {
        w.tx += step_tx;
        if (w.tx >= P.tiles_x) { w.tx -= P.tiles_x; ++w.ty; }
        w.ty += step_ty;
        if (w.ty >= P.tiles_y) { w.ty -= P.tiles_y; ++w.b; }
        w.b += step_b;
        if (++w.stage == nstages) { w.stage = 0; ++w.round; }
    };
    auto issue_k_tile = [&](const TileWalk& w) {
        const uint32_t base = smem_u32(smem + (size_t)w.stage * L.kstage_bytes);
        const uint32_t fb = bar(kBarKFull + w.stage);
        mbar_expect_tx(fb, (uint32_t)(6 * HW2 * 64 + 4 * P.TW * 64));
        tma_load_4d(base, &map_k, fb, h * kHeadDim, w.tx * P.TW - 1, w.ty * 4 - 1, w.b);
        tma_load_4d(base + L.halo_pad, &map_q, fb, h * kHeadDim, w.tx * P.TW, w.ty * 4, w.b);
    };
    auto issue_v_tile = [&](const TileWalk& w) {
        const uint32_t fb = bar(kBarVFull + w.stage);
        mbar_expect_tx(fb, (uint32_t)(6 * HW2 * 64));
        tma_load_4d(smem_u32(smem + L.v_off + (size_t)w.stage * L.halo_pad), &map_v, fb, h * kHeadDim,
                    w.tx * P.TW - 1, w.ty * 4 - 1, w.b);
    };

    // The fp32 weights of the head are staged in the LAST V stage's memory; that stage receives its
    // first tile only after every warp has finished with them.
    const unsigned char* w_stage = smem + L.v_off + (size_t)(SV - 1) * L.halo_pad;
    int k_issued = 0, v_issued = 0;                            // scheduler state (control warp, lane 0)
    TileWalk kq = walk_begin(), vq = kq;                       // next tile of the K queue / of the V queue
    if (my_tiles > 0 && warp == kCtlWarp && lane == 0) {
        mbar_expect_tx(bar(kBarWeights), 2 * kWeightBytes);
        bulk_load_1d(smem_u32(w_stage), P.wk + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
        bulk_load_1d(smem_u32(w_stage) + kWeightBytes, P.wv + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
        while (k_issued < my_tiles && k_issued < kKStages) { issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; }
        while (v_issued < my_tiles && v_issued < SV - 1) { issue_v_tile(vq); walk_next(vq, SV); ++v_issued; }
    }
    __syncwarp();

    bool ok = my_tiles > 0 && warp_wait(bar(kBarWeights), 0);
    const float* wks = reinterpret_cast<const float*>(w_stage);
    const float* wvs = wks + kHeadDim * 81;

    // ---- B tile of the value-side MMA: every thread converts its share ---------------------------
    if (ok) {
        unsigned char* sB = smem + L.b_off;
        for (int n = threadIdx.x; n < kBCols; n += kThreads) {     // one column (64 bytes of K) per thread
            unsigned char* col = sB + (n >> 3) * 512 + (n & 7) * 16;
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = 0u;
            if (n >= 288) {                                         // sum columns: 0 | 1 | 1 | 0,1,1,0..
#pragma unroll
                for (int i = 4; i < 12; ++i) w[i] = kOnesBf16x2;
                w[12] = pack_bf16(0.f, 1.f); w[13] = pack_bf16(1.f, 0.f);
            } else {
                const int ts = n >> 5, t = (ts % 3) * 3 + ts / 3;  // columns are ordered dx-major
                const int cn = n & 31, j = cn >> 3, wi = cn & 7;
                const float* wc = wvs + (8 * (wi >> 1) + 2 * j + (wi & 1)) * 81 + t;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int s0 = 2 * i, s1 = 2 * i + 1;
                    w[i] = pack_bf16(wc[s0 * 9] - (s0 == t ? 1.f : 0.f), wc[s1 * 9] - (s1 == t ? 1.f : 0.f));
                    const uint32_t oh = pack_bf16(s0 == t ? 1.f : 0.f, s1 == t ? 1.f : 0.f);
                    w[4 + i] = oh; w[8 + i] = oh;
                }
                const float o8 = t == 8 ? 1.f : 0.f;
                w[12] = pack_bf16(wc[72] - o8, o8); w[13] = pack_bf16(o8, 0.f);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4*>(col + c * 128) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
        }
        // key-side B fragments in fragment order: word (t, ks, lane, i) with n-tile i/2, register i%2
        uint32_t* sBk = reinterpret_cast<uint32_t*>(smem + L.bk_off);
        for (int w = threadIdx.x; w < 9 * 2 * 32 * 4; w += kThreads) {
            const int i = w & 3, ln = (w >> 2) & 31, ks = (w >> 7) & 1, t = w >> 8;
            const int fg = ln >> 2, ft = ln & 3, r = i & 1;
            const int c0 = 8 * ft + 4 * ks + 2 * r;
            uint32_t word;
            if ((i >> 1) == 0 || fg == 0) {                        // n-tile 0: slot fg; n-tile 1 column 0: slot 8
                const int sl = (i >> 1) == 0 ? fg : 8;
                const float e = (sl == t) ? 1.f : 0.f;
                word = pack_bf16(wks[c0 * 81 + sl * 9 + t] - e, wks[(c0 + 1) * 81 + sl * 9 + t] - e);
            } else {                                               // n-tile 1: column 1 sums tap 0, column n >= 2 tap n
                word = t == (fg == 1 ? 0 : fg) ? kOnesBf16x2 : 0u;
            }
            sBk[w] = word;
        }
        fence_proxy_async_smem();
    }
    __syncthreads();                                               // B tile and key-side fragments are complete

    if (warp >= kVWarps && warp < kCtlWarp) {
        // =====================================================================================
        // key warps
        // =====================================================================================
        const int kw = warp - kVWarps;
        const unsigned char* sBk = smem + L.bk_off + lane * 16;
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
            const int stage = ti % kKStages;
            if (!warp_wait(bar(kBarKFull + stage), (ti / kKStages) & 1)) { ok = false; break; }
            const int u0 = ti * U;
          for (int ul = (kw + kKWarps - u0 % kKWarps) % kKWarps; ul < U; ul += kKWarps) {
            const int u = u0 + ul;
            const int ux = ul * 8;
            const unsigned char* sK = smem + (size_t)stage * L.kstage_bytes;
            const unsigned char* sQ = sK + L.halo_pad;
            // q of the lane's four pixels (rows 0..3 of column ux + g)
            uint32_t qf[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = lds_u4(sQ, (uint32_t)(i * P.TW + ux + g) * 64u + tig * 16u);
                qf[i][0] = v.x; qf[i][1] = v.y; qf[i][2] = v.z; qf[i][3] = v.w;
            }
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
                for (int dy = 0; dy < 3; ++dy) {
                    const int t = dy * 3 + dx;
                    const uint4 b0 = lds_u4(sBk, (t * 2 + 0) * 512), b1 = lds_u4(sBk, (t * 2 + 1) * 512);
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        const uint4 k0 = kc[2 * mt + dy], k1 = kc[2 * mt + dy + 1];   // pixel rows 2mt / 2mt+1
                        uint32_t a0[4], a1[4];
                        a0[0] = hmul2_bf16(qf[2 * mt][0], k0.x);  a0[1] = hmul2_bf16(qf[2 * mt + 1][0], k1.x);
                        a0[2] = hmul2_bf16(qf[2 * mt][1], k0.y);  a0[3] = hmul2_bf16(qf[2 * mt + 1][1], k1.y);
                        a1[0] = hmul2_bf16(qf[2 * mt][2], k0.z);  a1[1] = hmul2_bf16(qf[2 * mt + 1][2], k1.z);
                        a1[2] = hmul2_bf16(qf[2 * mt][3], k0.w);  a1[3] = hmul2_bf16(qf[2 * mt + 1][3], k1.w);
                        mma_bf16(acc[mt][0], a0, b0.x, b0.y);
                        mma_bf16(acc[mt][1], a0, b0.z, b0.w);
                        mma_bf16(acc[mt][0], a1, b1.x, b1.y);
                        mma_bf16(acc[mt][1], a1, b1.z, b1.w);
                        if (t == 1) { mma_bf16(acc[mt][2], a0, ones_t1, ones_t1); mma_bf16(acc[mt][2], a1, ones_t1, ones_t1); }
                        if (t == 8) { mma_bf16(acc[mt][2], a0, ones_t8, ones_t8); mma_bf16(acc[mt][2], a1, ones_t8, ones_t8); }
                    }
                }
            }

            // unnormalised softmax weights; the 4 lanes of a quad share a pixel
            float e0[4], e1[4], e8[4];
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
            }

            // rows of the block's A tile: pixel i of column g is row 32*quadrant + 8*i + g
            const int blk = u >> 2, qd = u & 3, ab = blk % kABufs;
            if (!warp_wait(bar(kBarAFree + ab), ((blk / kABufs) & 1) ^ 1)) { ok = false; break; }
            unsigned char* sA = smem + L.a_off + ab * kABytes;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                unsigned char* row = sA + (4 * qd + i) * 512 + g * 16;
                const __nv_bfloat16 h0 = __float2bfloat16_rn(e0[i]), h1 = __float2bfloat16_rn(e1[i]);
                const uint32_t hi = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
                const uint32_t lo = pack_bf16(e0[i] - __bfloat162float(h0), e1[i] - __bfloat162float(h1));
                *reinterpret_cast<uint32_t*>(row + tig * 4) = hi;            // k 0..7   : meets D_v
                *reinterpret_cast<uint32_t*>(row + 128 + tig * 4) = hi;      // k 8..15  : meets [s == t]
                *reinterpret_cast<uint32_t*>(row + 256 + tig * 4) = lo;      // k 16..23 : meets [s == t]
                if (tig == 0) {
                    const __nv_bfloat16 h8 = __float2bfloat16_rn(e8[i]);
                    const float f8 = __bfloat162float(h8);
                    *reinterpret_cast<uint2*>(row + 384) = make_uint2(pack_bf16(f8, f8), pack_bf16(e8[i] - f8, 0.f));
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarAReady + ab));
          }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarKEmpty + stage)); // this warp is done with the stage
        }
    } else if (warp < kVWarps) {
        // =====================================================================================
        // value warps (warp index = quadrant of the block = TMEM lanes 32*warp ..)
        // =====================================================================================
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarWeightsDone));
        const int qd = warp & 3, half = warp >> 2;                 // quadrant; which blocks (even / odd)
        const uint32_t tq = tmem + ((uint32_t)(32 * qd) << 16);

        TileWalk vw = walk_begin();
        for (int ti = 0; ok && ti < my_tiles; ++ti, walk_next(vw, SV)) {
            const int tx = vw.tx, ty = vw.ty, b = vw.b, stage = vw.stage;
            if (!warp_wait(bar(kBarVFull + stage), vw.round & 1)) { ok = false; break; }
            const int u0 = ti * U;
          for (int ul = (qd + 4 - u0 % 4) % 4; ul < U; ul += 4) {
            const int u = u0 + ul;
            if (((u >> 2) & 1) != half) continue;                  // the other warp of this quadrant takes it
            const int ux = ul * 8;
            const int blk = u >> 2;
            const unsigned char* sV = smem + L.v_off + (size_t)stage * L.halo_pad;
            const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;

            float o_acc[4][8];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int c = 0; c < 8; ++c) o_acc[i][c] = 0.f;
            float inv[4] = {0.f, 0.f, 0.f, 0.f};

#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                const int cs = 3 * (blk >> 1) + dx, ds = 2 * half + (cs & 1);   // chunk index within the set, TMEM slot
                if (!warp_wait(bar(kBarDFull + ds), (cs >> 1) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t colbase = ds * kDSlotCols;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    // A'[pixel rows 2mt, 2mt+1][taps (dy = 0..2, dx)][8 channels]: three loads in flight
                    // while the halo rows 2mt .. 2mt+3 of column dx come out of shared memory
                    uint32_t dr[48];
                    const uint32_t ta = tq + ((uint32_t)(16 * mt) << 16) + colbase;
                    tmem_ld3_16x256b_x4_nowait(ta, ta + 32, ta + 64, dr);
                    uint4 vp[4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) vp[r] = lds_u4(sV, off0 + (uint32_t)((2 * mt + r) * HW2 + dx) * 64u);
                    float vf[4][8];                                // widened to fp32
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const uint4 v = vp[r];
                        vf[r][0] = bf16_lo(v.x); vf[r][1] = bf16_hi(v.x);
                        vf[r][2] = bf16_lo(v.y); vf[r][3] = bf16_hi(v.y);
                        vf[r][4] = bf16_lo(v.z); vf[r][5] = bf16_hi(v.z);
                        vf[r][6] = bf16_lo(v.w); vf[r][7] = bf16_hi(v.w);
                    }
                    tmem_wait_ld48(dr);
                    float d[48];
#pragma unroll
                    for (int i = 0; i < 48; ++i) d[i] = __uint_as_float(dr[i]);
#pragma unroll
                    for (int dy = 0; dy < 3; ++dy) {               // halo rows dy (half 0) and dy+1 (half 1)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            ffma2(o_acc[2 * mt][2 * j], o_acc[2 * mt][2 * j + 1], d[16 * dy + 4 * j], d[16 * dy + 4 * j + 1],
                                  vf[dy][2 * j], vf[dy][2 * j + 1]);
                            ffma2(o_acc[2 * mt + 1][2 * j], o_acc[2 * mt + 1][2 * j + 1], d[16 * dy + 4 * j + 2], d[16 * dy + 4 * j + 3],
                                  vf[dy + 1][2 * j], vf[dy + 1][2 * j + 1]);
                        }
                    }
                }
                if (dx == 2) {                                     // sum_s e[p,s] of the four pixels
                    float s0[4], s1[4];
                    tmem_ld_16x256b_x1(tq + colbase + 96, s0);                      // pixel rows 0, 1
                    tmem_ld_16x256b_x1(tq + (16u << 16) + colbase + 96, s1);        // pixel rows 2, 3
                    inv[0] = rcp_approx(s0[0]); inv[1] = rcp_approx(s0[2]); inv[2] = rcp_approx(s1[0]); inv[3] = rcp_approx(s1[2]);
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarDFree + ds));
            }
            if (!ok) break;

            {
                const int x = tx * P.TW + ux + g, y0 = ty * 4;
                __nv_bfloat16* op = P.out + ((size_t)(b * P.H + y0) * P.W + x) * C + h * kHeadDim + tig * 8;
                const size_t row_stride = (size_t)P.W * C;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (x < P.W && y0 + i < P.H) {
                        uint4 r;
                        r.x = pack_bf16(o_acc[i][0] * inv[i], o_acc[i][1] * inv[i]);
                        r.y = pack_bf16(o_acc[i][2] * inv[i], o_acc[i][3] * inv[i]);
                        r.z = pack_bf16(o_acc[i][4] * inv[i], o_acc[i][5] * inv[i]);
                        r.w = pack_bf16(o_acc[i][6] * inv[i], o_acc[i][7] * inv[i]);
                        *reinterpret_cast<uint4*>(op + i * row_stride) = r;
                    }
                }
            }
          }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarVEmpty + stage)); // this warp is done with the stage
        }
        // quadrants of the last block that hold no unit: keep the chunk barriers in step
        if (ok && my_blocks > 0 && (my_units & 3) != 0 && qd >= (my_units & 3) && ((my_blocks - 1) & 1) == half) {
            for (int dx = 0; ok && dx < 3; ++dx) {
                const int cs = 3 * ((my_blocks - 1) >> 1) + dx, ds = 2 * half + (cs & 1);
                if (!warp_wait(bar(kBarDFull + ds), (cs >> 1) & 1)) { ok = false; break; }
                if (lane == 0) mbar_arrive(bar(kBarDFree + ds));
            }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarVDone));
    } else {
        // =====================================================================================
        // control warp: lane 0 issues the value-side MMAs; the warp owns tensor memory
        // =====================================================================================
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarWeightsDone));
        if (lane == 0 && ok) {
            // One thread runs both queues by polling, so neither can hold up the other:
            //   TMA queue: tile n goes out as soon as its stage is free;
            //   MMA queue: chunk (blk, dx) goes out as soon as the block's A tile is complete and
            //   its TMEM slot has been read.
            // It gives up when nothing has moved for about two seconds.
            const uint32_t sA0 = smem_u32(smem + L.a_off), sB0 = smem_u32(smem + L.b_off);
            // Every pass first puts all its barrier tests in flight together and only then acts on
            // them: this thread shares its scheduler with three busy warps, and tests taken one
            // after the other, each behind a branch, made a pass cost as much as a whole chunk.
            bool weights_done = false;
            int blk0 = 0, blk1 = 1, dx0 = 0, dx1 = 0;                // MMA queue of each value-warp set
            bool stood_in = false;
            const int partial = (my_units & 3) != 0 ? my_blocks - 1 : -1;   // block with fewer than 4 units
            int left = 2 * my_tiles - k_issued - v_issued + 3 * my_blocks;  // actions still to issue
            uint32_t idle = 0;
            auto issue_chunk = [&](int set, int& blk, int& dx) {
                const int ab = blk % kABufs, cs = 3 * (blk >> 1) + dx, ds = 2 * set + (cs & 1);
                tc_fence_after_sync();
                // columns dx*96 .. of B; K = 32 = two instructions of K = 16 (256 bytes apart)
                const uint32_t sA = sA0 + ab * kABytes, sB = sB0 + dx * 12 * 512;
                const uint32_t idesc = dx == 2 ? kIdesc112 : kIdesc96;
                const uint32_t dcol = tmem + ds * kDSlotCols;
                umma_bf16_ss(dcol, umma_smem_desc(sA, 128, 512), umma_smem_desc(sB, 128, 512), idesc, 0);
                umma_bf16_ss(dcol, umma_smem_desc(sA + 256, 128, 512), umma_smem_desc(sB + 256, 128, 512), idesc, 1);
                umma_commit(bar(kBarDFull + ds));
                if (dx == 2) { umma_commit(bar(kBarAFree + ab)); dx = 0; blk += 2; }
                else ++dx;
                --left;
            };
            while (left > 0) {
                if (!weights_done) weights_done = mbar_test(bar(kBarWeightsDone), 0);
                if (!stood_in && (blk0 == partial || blk1 == partial)) {
                    // partial last block: stand in for the units that do not exist.  A queue has
                    // reached this block, so the previous phase of its AReady barrier is over.
                    for (int m = my_units & 3; m < 4; ++m) mbar_arrive(bar(kBarAReady + partial % kABufs));
                    stood_in = true;
                }
                // A stage or slot in its first round is free: parity 1 of a fresh barrier tests true.
                const int cs0 = 3 * (blk0 >> 1) + dx0, cs1 = 3 * (blk1 >> 1) + dx1;
                const uint32_t tK = mbar_test_u32(bar(kBarKEmpty + kq.stage), (kq.round - 1) & 1);
                const uint32_t tV = mbar_test_u32(bar(kBarVEmpty + vq.stage), (vq.round - 1) & 1);
                const uint32_t tA0 = mbar_test_u32(bar(kBarAReady + blk0 % kABufs), (blk0 / kABufs) & 1);
                const uint32_t tD0 = mbar_test_u32(bar(kBarDFree + (cs0 & 1)), ((cs0 >> 1) & 1) ^ 1);
                const uint32_t tA1 = mbar_test_u32(bar(kBarAReady + blk1 % kABufs), (blk1 / kABufs) & 1);
                const uint32_t tD1 = mbar_test_u32(bar(kBarDFree + 2 + (cs1 & 1)), ((cs1 >> 1) & 1) ^ 1);
                const int left_before = left;
                if (tK != 0 && k_issued < my_tiles) {
                    issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; --left;
                }
                // the last V stage held the weights: its first tile waits until every warp is done with them
                if (tV != 0 && v_issued < my_tiles && (v_issued != SV - 1 || weights_done)) {
                    issue_v_tile(vq); walk_next(vq, SV); ++v_issued; --left;
                }
                if ((tA0 & tD0) != 0 && blk0 < my_blocks) issue_chunk(0, blk0, dx0);
                if ((tA1 & tD1) != 0 && blk1 < my_blocks) issue_chunk(1, blk1, dx1);
                if (left != left_before) idle = 0;
                else if (++idle > (1u << 24)) { ok = false; break; }      // nothing moved for seconds: give up
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        // tensor memory is released once the value warps have stopped reading it (or given up)
        if (my_tiles > 0 && !warp_wait(bar(kBarVDone), 0)) ok = false;
        tc_fence_after_sync();
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
    if (!ok && my_tiles > 0 && lane == 0) atomicExch(P.status, 1);
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

bool umma_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && ksize == 3;
}

cudaError_t umma_setup() {
    if (!encode_fn()) return cudaErrorNotSupported;
    return cudaFuncSetAttribute(umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

cudaError_t launch_umma(const Problem& p, int* d_status, int num_sms, cudaStream_t stream) {
    // tile width: a multiple of 8 up to 64, splitting the row evenly
    const int txn = (p.W + 63) / 64;
    const int TW = ((((p.W + txn - 1) / txn) + 7) / 8) * 8;
    UmmaParams P;
    P.wk = p.wk; P.wv = p.wv; P.bias = p.bias;
    P.out = static_cast<__nv_bfloat16*>(p.out);
    P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.TW = TW;
    P.tiles_x = (p.W + TW - 1) / TW;
    P.tiles_y = (p.H + 3) / 4;
    P.stages = 2;                                          // V ring depth: as deep as fits
    for (int st = kMaxVStages; st >= 2; --st)
        if (smem_layout(TW, st).total <= kMaxSmem) { P.stages = st; break; }
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
    umma_kernel<<<grid, kThreads, L.total, stream>>>(map_q, map_k, map_v, P);
    return cudaGetLastError();
}

}  // namespace slide_attn
