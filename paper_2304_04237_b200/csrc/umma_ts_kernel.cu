// UMMA_TS variant (bf16, head_dim 32, k = 3): BOTH contractions of the fused forward on the
// 5th-generation tensor core (tcgen05.mma), each with its A operand in tensor memory, so neither the
// q.k products nor the softmax weights pass through shared memory.
//
// Arithmetic (Eq. 2 with Eq. 12 inside; w = E + D, E the one-hot shift of Eq. 11):
//   product warps   P[p,(t,c)] = q[p,c] k[p+off(t),c]   packed bf16 multiply -> tcgen05.st (TMEM)
//   key MMA         L[p,n]     = sum_{t,c} P[p,(t,c)] Bk[(t,c),n]       tcgen05.mma, A from TMEM
//                   n = 0..8: deformed part D_k of slot n;  n = 9..17: plain q.k sum of tap n-9
//   product warps   logit[s] = (L[s] + L[9+s]) scale + bias[s];  e = exp2(logit - max) / sum_s exp2(logit - max)
//                   (tcgen05.ld.32x32b: one thread holds all logits of one pixel, no shuffles)
//                   A' row = e_hi | e_hi | e_lo | e8_hi e8_hi e8_lo 0..   -> tcgen05.st (TMEM)
//   value MMA       D[p,(t,c)] = sum_k A'[p,k] Bv[k,(t,c)]                     A from TMEM
//   value warps     out[p,c] = sum_t D[p,t,c] v[p+off(t),c]
//
// Tensor memory (512 columns): two value-chunk slots 112 columns apart, 96 used (chunk c = 3 blk + dx -> slot
// c & 1), four P chunks of 48 (3 taps x 32 bf16, chunk -> buffer c & 3), two logit tiles of 32, two A' tiles of 16.
//
// Warps (20, 86 registers): 0-7 value warps (quadrant = warp % 4, pixel-row pair = warp / 4, every
// block), 8-15 product warps (quadrant, pixel-row pair: P of their 16 pixels of every block; the
// softmax of a block is done for the whole quadrant by the warp whose pair index equals the block's
// parity, after it has stored the P of the next block), 16 and 18 key-side control (the 18 key MMAs
// of the even / odd blocks, taking turns through two barriers so that the P-ready barriers are
// waited on strictly in chunk order), 17 value-side control
// (value MMAs), 19 TMA thread (K/q and V rings).  The MMA threads have one thing to wait for at a
// time and park in mbarrier waits instead of polling: that alone was worth 10 % of the kernel time.
// Warp 16 owns tensor memory.  Every wait is bounded; a wait that runs out sets the status word, and
// tensor memory is released on every path.
//
// What bounds it: instruction issue on the CUDA cores.  An M = 128 MMA costs about N / 2 cycles (18 of N = 32 and
// 6 of N = 96 per 128 pixels: 540 cycles of a block period of about 2 850), the value warps are busy from block to
// block, everything else waits for them, and with four or five warps per scheduler the time follows the instruction
// count (5.9 k warp instructions per block: the q.k products, the widenings of V, the accumulator x V multiply-adds).
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

// Time-line build (-DSLIDE_ATTN_TIMELINE): CTA 0 stamps clock64 around the waits of one warp of every role, per
// chunk (c = 3 block + dx) or block; slide_attn_umma_ts_timeline copies the stamps out.  The stamps skip no work;
// the library proper is built without them.
#ifdef SLIDE_ATTN_TIMELINE
__device__ long long g_umma_timeline[16][128];
#define UMMA_TL(role, idx) do { if (blockIdx.x == 0 && (idx) < 128) g_umma_timeline[role][idx] = clock64(); } while (0)
#else
#define UMMA_TL(role, idx) do {} while (0)
#endif

namespace {

constexpr int kHeadDim = 32;
constexpr int kVWarps = 8;
constexpr int kPWarps = 8;
constexpr int kCtlK = kVWarps + kPWarps;                // warp 16: key MMAs of the even blocks, TMEM owner
constexpr int kCtlV = kCtlK + 1;                        // warp 17: value MMAs
constexpr int kCtlK2 = kCtlV + 1;                       // warp 18: key MMAs of the odd blocks
constexpr int kCtlT = kCtlK2 + 1;                       // warp 19: TMA thread, K/q and V tiles
constexpr int kThreads = (kCtlT + 1) * 32;
constexpr int kKStages = 2;
constexpr int kMaxVStages = 4;
constexpr int kBCols = 288;                             // value columns: (tap, channel)
constexpr int kBBytes = kBCols * 64;
constexpr int kBkBytes = 36 * 512;                      // key-side B: 288 K x 32 N bf16
constexpr int kImgBytes = kBBytes + kBkBytes;           // both B images of one head, as the prep kernel leaves them
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kTmemCols = 512;
// tensor-memory columns
constexpr uint32_t kColD = 0;                           // two value-chunk slots of 112 columns (chunk c -> slot c & 1)
constexpr uint32_t kColP = 224;                         // four P chunks of 48 columns (3 taps x 32 bf16)
constexpr uint32_t kColL = 416;                         // two logit tiles of 32 columns
constexpr uint32_t kColE = 480;                         // two A' tiles of 16 columns (32 bf16)
constexpr uint32_t kIdesc96 = umma_idesc_bf16(128, 96);
constexpr uint32_t kIdesc32 = umma_idesc_bf16(128, 32);

struct UmmaParams {
    const unsigned char* bimg;       // per head: value-side B image (kBBytes) then key-side B image (kBkBytes)
    const float* bias;
    __nv_bfloat16* out;
    int* status;
    int B, H, W, heads;
    int tiles_x, tiles_y;
    float scale_log2e;
};

struct Smem {
    uint32_t halo_pad, kstage_bytes, v_off, b_off, bk_off, tmem_off, bar_off, total;
};

__host__ __device__ constexpr Smem smem_layout(int TW, int vstages) {
    Smem s{};
    s.halo_pad = ((uint32_t)(6 * (TW + 2) * 64) + 1023u) & ~1023u;
    s.kstage_bytes = s.halo_pad + (((uint32_t)(4 * TW * 64) + 1023u) & ~1023u);
    s.v_off = kKStages * s.kstage_bytes;
    s.b_off = s.v_off + vstages * s.halo_pad;
    s.bk_off = s.b_off + kBBytes;
    s.tmem_off = s.bk_off + kBkBytes;
    s.bar_off = s.tmem_off + 16;
    s.total = s.bar_off + 40 * 8 + 1024;
    return s;
}

constexpr size_t kMaxSmem = 227 * 1024;

// V stages that fit beside everything else for a tile width (the kernel is instantiated per width,
// so that every shared-memory offset and stride is a compile-time constant)
__host__ __device__ constexpr int v_stages_for(int TW) {
    for (int st = kMaxVStages; st >= 2; --st)
        if (smem_layout(TW, st).total <= kMaxSmem) return st;
    return 0;
}

constexpr int kBarKFull = 0;         // [2]
constexpr int kBarKEmpty = 2;        // [2]  count 8 (product warps)
constexpr int kBarVFull = 4;         // [4]
constexpr int kBarVEmpty = 8;        // [4]  count 8
constexpr int kBarWeights = 12;      // both B images have landed (one bulk copy)
constexpr int kBarPReady = 14;       // [4]  count 8: P chunk stored by the eight product warps
constexpr int kBarPFree = 18;        // [4]  key MMAs reading the chunk are complete
constexpr int kBarLFull = 22;        // [2]  logits of a block complete
constexpr int kBarLFree = 24;        // [2]  count 4: logits read (one product warp per quadrant)
constexpr int kBarEReady = 26;       // [2]  count 4: A' rows stored
constexpr int kBarEFree = 28;        // [2]  value MMAs of the block complete
constexpr int kBarDFull = 30;        // [2]  value chunk complete
constexpr int kBarDFree = 32;        // [2]  count 8: value chunk read
constexpr int kBarVDone = 34;        // count 8
constexpr int kBarTurn = 35;         // [2]  the other key-control thread has taken the last chunk of its block

__device__ __forceinline__ uint4 lds_u4(const unsigned char* base, uint32_t off) {
    return *reinterpret_cast<const uint4*>(base + off);
}
// Hand-offs of tensor memory between threads: the side that has read or written TMEM issues
// tcgen05.wait::ld / ::st (the accesses are then complete) and arrives on an mbarrier; the side that
// takes over waits on it and issues tcgen05.fence::after_thread_sync before its own tcgen05 work.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}

// ---------------------------------------------------------------------------------------------
// Prep kernel: the two B images of every head, in the shared-memory layout the MMAs read
// (K-major core matrices of 8 rows x 16 bytes, no swizzle), written to the context workspace once per
// forward.  Block (h, part) builds a share of head h's items.
//   value side  [288 columns][32 K] bf16: column n = (tap-column-major tap, channel); K rows
//               0..7 D_v[c][s][t], 8..15 and 16..23 the one-hot [s = t], 24 D_v[c][8][t], 25, 26 [t = 8]
//               (the A' row is e_hi | e_hi | e_lo | e8_hi e8_hi e8_lo)
//   key side    [288 K][32 N] bf16: K = 32 tap + kappa (kappa -> channel as tcgen05.st lays P out),
//               N 0..8 D_k[c][n][t], 9..17 the one-hot [n - 9 = t]
__global__ void __launch_bounds__(256)
umma_ts_prep_kernel(const float* __restrict__ wk, const float* __restrict__ wv, unsigned char* __restrict__ img)
{
    grid_launch_dependents();        // the main kernel may start its own prologue now
    const int h = blockIdx.x;
    const float* wks = wk + (size_t)h * kHeadDim * 81;
    const float* wvs = wv + (size_t)h * kHeadDim * 81;
    unsigned char* sB = img + (size_t)h * kImgBytes;
    unsigned char* sBk = sB + kBBytes;
    for (int item = blockIdx.y * blockDim.x + threadIdx.x; item < kBCols + 36 * 32; item += gridDim.y * blockDim.x) {
        if (item < kBCols) {
            const int n = item;
            unsigned char* col = sB + (n >> 3) * 512 + (n & 7) * 16;
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = 0u;
            {
                const int ts = n >> 5, t = (ts % 3) * 3 + ts / 3;
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
        } else {
            const int it = item - kBCols;
            const int n = it & 31, kg = it >> 5;
            const int t = kg >> 2, kap0 = (kg & 3) * 8;
            float val[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int kap = kap0 + e;
                const int c = 8 * ((kap & 15) >> 2) + (kap & 3) + (kap >= 16 ? 4 : 0);
                float x = 0.f;
                if (n < 9) x = wks[c * 81 + n * 9 + t] - (n == t ? 1.f : 0.f);
                else if (n < 18) x = (n - 9 == t) ? 1.f : 0.f;
                val[e] = x;
            }
            *reinterpret_cast<uint4*>(sBk + kg * 512 + (n >> 3) * 128 + (n & 7) * 16) =
                make_uint4(pack_bf16(val[0], val[1]), pack_bf16(val[2], val[3]), pack_bf16(val[4], val[5]), pack_bf16(val[6], val[7]));
        }
    }
}

template <int TW>
__global__ void __launch_bounds__(kThreads, 1)
umma_ts_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
             const __grid_constant__ CUtensorMap map_v, const UmmaParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int SV = v_stages_for(TW);
    constexpr Smem L = smem_layout(TW, SV);
    const uint32_t bar0 = smem_u32(smem + L.bar_off);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    // the warp index through a shuffle: the compiler then knows it is the same in every lane
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    constexpr int U = TW >> 3;
    constexpr int HW2 = TW + 2;

    const int h = blockIdx.x % P.heads;
    const int rank = blockIdx.x / P.heads;
    const int nrank = ((int)gridDim.x - h + P.heads - 1) / P.heads;
    const int tiles_per_head = P.B * P.tiles_y * P.tiles_x;
    // tiles are dealt round-robin: neighbouring CTAs work on neighbouring tiles at the same time, which
    // keeps the halos they share in L2
    const int my_tiles = rank < tiles_per_head ? (tiles_per_head - rank + nrank - 1) / nrank : 0;
    const int my_units = my_tiles * U;
    const int my_blocks = (my_units + 3) >> 2;
    const int C = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kKStages; ++s) { mbar_init_only(bar(kBarKFull + s), 1); mbar_init_only(bar(kBarKEmpty + s), kPWarps); }
        for (int s = 0; s < kMaxVStages; ++s) { mbar_init_only(bar(kBarVFull + s), 1); mbar_init_only(bar(kBarVEmpty + s), kVWarps); }
        mbar_init_only(bar(kBarWeights), 1);
        for (int i = 0; i < 4; ++i) { mbar_init_only(bar(kBarPReady + i), kPWarps); mbar_init_only(bar(kBarPFree + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init_only(bar(kBarLFull + i), 1);
            mbar_init_only(bar(kBarLFree + i), 4);
            mbar_init_only(bar(kBarEReady + i), 4);
            mbar_init_only(bar(kBarEFree + i), 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init_only(bar(kBarDFull + i), 1); mbar_init_only(bar(kBarDFree + i), kVWarps); }
        mbar_init_only(bar(kBarVDone), kVWarps);
        mbar_init_only(bar(kBarTurn + 0), 1);
        mbar_init_only(bar(kBarTurn + 1), 1);
        mbar_init_fence();
    }
    if (warp == kCtlK) tmem_alloc(smem_u32(smem + L.tmem_off), kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<const volatile uint32_t*>(smem + L.tmem_off);

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
        mbar_expect_tx(fb, (uint32_t)(6 * HW2 * 64 + 4 * TW * 64));
        tma_load_4d(base, &map_k, fb, h * kHeadDim, w.tx * TW - 1, w.ty * 4 - 1, w.b);
        tma_load_4d(base + L.halo_pad, &map_q, fb, h * kHeadDim, w.tx * TW, w.ty * 4, w.b);
    };
    auto issue_v_tile = [&](const TileWalk& w) {
        const uint32_t fb = bar(kBarVFull + w.stage);
        mbar_expect_tx(fb, (uint32_t)(6 * HW2 * 64));
        tma_load_4d(smem_u32(smem + L.v_off + (size_t)w.stage * L.halo_pad), &map_v, fb, h * kHeadDim,
                    w.tx * TW - 1, w.ty * 4 - 1, w.b);
    };

    // The B images of this CTA's head were laid out by the prep kernel of the same forward; they come
    // in with one bulk copy, sent for together with the first K/q and V tiles.  Only the MMA threads
    // wait for them.  The prep kernel may still be running when this kernel starts (programmatic
    // dependent launch), so the thread that reads its output waits for that grid first; nothing
    // else in this kernel depends on it.
    int k_issued = 0, v_issued = 0;
    TileWalk kq = walk_begin(), vq = kq;
    if (my_tiles > 0 && warp == kCtlT) {
        // the same lane is elected here and in the refill loop below (the election is deterministic for
        // a given member mask), so the ring positions it advances here are the ones it continues from
        uint32_t leader;
        if (elect_one(leader)) {
            while (k_issued < my_tiles && k_issued < kKStages) { issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; }
            while (v_issued < my_tiles && v_issued < SV) { issue_v_tile(vq); walk_next(vq, SV); ++v_issued; }
        }
    }
    if (my_tiles > 0 && warp == kCtlV && lane == 0) {
        grid_dependency_wait();
        mbar_expect_tx(bar(kBarWeights), kImgBytes);
        bulk_load_1d(smem_u32(smem + L.b_off), P.bimg + (size_t)h * kImgBytes, kImgBytes, bar(kBarWeights));
    }
    __syncwarp();
    bool ok = my_tiles > 0;

    if (warp >= kVWarps && warp < kCtlK) {
        // =====================================================================================
        // product warps: warp (q, pm) takes pixel rows 2pm, 2pm+1 of unit 4 blk + q of every block
        // =====================================================================================
        const int q = (warp - kVWarps) & 3;                        // == warp % 4
        const int pm = (warp - kVWarps) >> 2;                      // pixel-row pair of the unit; softmax of blocks = pm mod 2
        const uint32_t tq = tmem + ((uint32_t)(32 * q) << 16);
        float biasl[9];
#pragma unroll
        for (int s = 0; s < 9; ++s) biasl[s] = P.bias ? P.bias[h * 9 + s] * kLog2e : 0.f;

        // softmax of block sb (thread = pixel = TMEM lane 32 q + lane); `valid`: the unit exists
        auto softmax_block = [&](int sb, bool valid) -> bool {
            const int lb = sb & 1;
            if (warp == kVWarps && lane == 0) UMMA_TL(3, sb);              // softmax of block sb: before the logits wait
            if (!warp_wait(bar(kBarLFull + lb), (sb >> 1) & 1)) return false;
            if (warp == kVWarps && lane == 0) UMMA_TL(4, sb);
            tc_fence_after_sync();
            float Lg[32];
            tmem_ld_32x32b_x32(tq + kColL + 32 * lb, Lg);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarLFree + lb));
            uint32_t row[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) row[i] = 0u;
            if (valid) {
                float l[9], m = -INFINITY;
#pragma unroll
                for (int s = 0; s < 9; ++s) { l[s] = (Lg[s] + Lg[9 + s]) * P.scale_log2e + biasl[s]; m = fmaxf(m, l[s]); }
                float e[9], sum = 0.f;
#pragma unroll
                for (int s = 0; s < 9; ++s) { e[s] = fast_exp2(l[s] - m); sum += e[s]; }
                const float inv = rcp_approx(sum);               // the weights leave normalised: the value side only sums
                float hi[9], lo[9];
#pragma unroll
                for (int s = 0; s < 9; ++s) {
                    const float a = e[s] * inv;
                    hi[s] = __bfloat162float(__float2bfloat16_rn(a));
                    lo[s] = a - hi[s];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    row[i] = pack_bf16(hi[2 * i], hi[2 * i + 1]);
                    row[4 + i] = row[i];
                    row[8 + i] = pack_bf16(lo[2 * i], lo[2 * i + 1]);
                }
                row[12] = pack_bf16(hi[8], hi[8]);
                row[13] = pack_bf16(lo[8], 0.f);
            }
            if (warp == kVWarps && lane == 0) UMMA_TL(5, sb);              // weights computed: before the A'-free wait
            if (!warp_wait(bar(kBarEFree + lb), ((sb >> 1) & 1) ^ 1)) return false;
            if (warp == kVWarps && lane == 0) UMMA_TL(6, sb);
            tc_fence_after_sync();
            tmem_st_32x32b_x16(tq + kColE + 16 * lb, row);
            tmem_wait_st();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEReady + lb));
            return true;
        };

        int done_blocks = 0;                                       // blocks whose P this warp has delivered
        int next_sm = pm;                                          // next block whose softmax is this warp's
        // softmax of this warp's blocks below `upto`
        auto softmax_upto = [&](int upto) -> bool {
            while (next_sm < upto) {
                if (!softmax_block(next_sm, 4 * next_sm + q < my_units)) return false;
                next_sm += 2;
            }
            return true;
        };
        for (int ti = 0; ok && ti < my_tiles; ++ti) {
            const int stage = ti % kKStages;
            if (!warp_wait(bar(kBarKFull + stage), (ti / kKStages) & 1)) { ok = false; break; }
            const int u0 = ti * U;
            for (int ul = (q + 4 - u0 % 4) % 4; ul < U; ul += 4) {
                const int u = u0 + ul, blk = u >> 2;
                const int ux = ul * 8;
                const unsigned char* sK = smem + (size_t)stage * L.kstage_bytes;
                const unsigned char* sQ = sK + L.halo_pad;
                uint32_t qf[2][4];                                 // pixel rows 2pm, 2pm+1 of column ux + g
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint4 v = lds_u4(sQ, (uint32_t)((2 * pm + i) * TW + ux + g) * 64u + tig * 16u);
                    qf[i][0] = v.x; qf[i][1] = v.y; qf[i][2] = v.z; qf[i][3] = v.w;
                }
                const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;
#pragma unroll
                for (int dx = 0; dx < 3; ++dx) {
                    const int pc = 3 * blk + dx, pb = pc & 3;
                    uint4 kc[4];                                   // halo rows 2pm .. 2pm+3 of column dx
#pragma unroll
                    for (int r = 0; r < 4; ++r) kc[r] = lds_u4(sK, off0 + (uint32_t)((2 * pm + r) * HW2 + dx) * 64u);
                    if (warp == kVWarps && lane == 0) UMMA_TL(0, pc);      // product warp (0, 0): before the P-free wait
                    if (!warp_wait(bar(kBarPFree + pb), ((pc >> 2) & 1) ^ 1)) { ok = false; break; }
                    if (warp == kVWarps && lane == 0) UMMA_TL(1, pc);      // after it
                    tc_fence_after_sync();
#pragma unroll
                    for (int dy = 0; dy < 3; ++dy) {
                        const uint4 k0 = kc[dy], k1 = kc[dy + 1];
                        uint32_t r[8];
                        r[0] = hmul2_bf16(qf[0][0], k0.x); r[1] = hmul2_bf16(qf[0][1], k0.y);
                        r[2] = hmul2_bf16(qf[1][0], k1.x); r[3] = hmul2_bf16(qf[1][1], k1.y);
                        r[4] = hmul2_bf16(qf[0][2], k0.z); r[5] = hmul2_bf16(qf[0][3], k0.w);
                        r[6] = hmul2_bf16(qf[1][2], k1.z); r[7] = hmul2_bf16(qf[1][3], k1.w);
                        tmem_st_16x256b_x2(tq + ((uint32_t)(16 * pm) << 16) + kColP + 48 * pb + 16 * dy, r);
                    }
                    tmem_wait_st();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarPReady + pb));
                    if (warp == kVWarps && lane == 0) UMMA_TL(2, pc);      // chunk delivered
                }
                if (!ok) break;
                ++done_blocks;
                // the logits of the blocks before this one are complete by now (or soon)
                if (!softmax_upto(blk)) { ok = false; break; }
            }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarKEmpty + stage));
        }
        // a quadrant the last block lacks: deliver its (empty) share so that the counts complete
        if (ok && done_blocks < my_blocks) {
            const int blk = my_blocks - 1;
            for (int dx = 0; ok && dx < 3; ++dx) {
                const int pc = 3 * blk + dx, pb = pc & 3;
                if (!warp_wait(bar(kBarPFree + pb), ((pc >> 2) & 1) ^ 1)) { ok = false; break; }
                if (lane == 0) mbar_arrive(bar(kBarPReady + pb));
            }
        }
        if (ok && !softmax_upto(my_blocks)) ok = false;
    } else if (warp < kVWarps) {
        // =====================================================================================
        // value warps: warp (qd, m) takes pixel rows 2m, 2m+1 of quadrant qd of every block
        // =====================================================================================
        const int qd = warp & 3, m = warp >> 2;
        const uint32_t tq = tmem + ((uint32_t)(32 * qd + 16 * m) << 16);

        TileWalk vw = walk_begin();
        for (int ti = 0; ok && ti < my_tiles; ++ti, walk_next(vw, SV)) {
            const int tx = vw.tx, ty = vw.ty, b = vw.b, stage = vw.stage;
            if (!warp_wait(bar(kBarVFull + stage), vw.round & 1)) { ok = false; break; }
            const int u0 = ti * U;
          for (int ul = (qd + 4 - u0 % 4) % 4; ul < U; ul += 4) {
            const int u = u0 + ul;
            const int ux = ul * 8;
            const int blk = u >> 2;
            const unsigned char* sV = smem + L.v_off + (size_t)stage * L.halo_pad;
            const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;

            float o_acc[2][8];
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int c = 0; c < 8; ++c) o_acc[i][c] = 0.f;

#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
                const int cs = 3 * blk + dx, ds = cs & 1;
                if (warp == 0 && lane == 0) UMMA_TL(7, cs);                // value warp (0, 0): before the chunk wait
                if (!warp_wait(bar(kBarDFull + ds), (cs >> 1) & 1)) { ok = false; break; }
                if (warp == 0 && lane == 0) UMMA_TL(8, cs);
                tc_fence_after_sync();
                const uint32_t colbase = kColD + ds * 112;
                {
                    uint32_t dr[48];
                    const uint32_t ta = tq + colbase;
                    tmem_ld3_16x256b_x4_nowait(ta, ta + 32, ta + 64, dr);
                    uint4 vp[4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) vp[r] = lds_u4(sV, off0 + (uint32_t)((2 * m + r) * HW2 + dx) * 64u);
                    float vf[4][8];
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
                    for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            ffma2(o_acc[0][2 * j], o_acc[0][2 * j + 1], d[16 * dy + 4 * j], d[16 * dy + 4 * j + 1],
                                  vf[dy][2 * j], vf[dy][2 * j + 1]);
                            ffma2(o_acc[1][2 * j], o_acc[1][2 * j + 1], d[16 * dy + 4 * j + 2], d[16 * dy + 4 * j + 3],
                                  vf[dy + 1][2 * j], vf[dy + 1][2 * j + 1]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarDFree + ds));
                if (warp == 0 && lane == 0) UMMA_TL(9, cs);                // chunk consumed
            }
            if (!ok) break;

            {
                const int x = tx * TW + ux + g, y0 = ty * 4 + 2 * m;
                __nv_bfloat16* op = P.out + ((size_t)(b * P.H + y0) * P.W + x) * C + h * kHeadDim + tig * 8;
                const size_t row_stride = (size_t)P.W * C;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    if (x < P.W && y0 + i < P.H) {
                        uint4 r;
                        r.x = pack_bf16(o_acc[i][0], o_acc[i][1]);
                        r.y = pack_bf16(o_acc[i][2], o_acc[i][3]);
                        r.z = pack_bf16(o_acc[i][4], o_acc[i][5]);
                        r.w = pack_bf16(o_acc[i][6], o_acc[i][7]);
                        *reinterpret_cast<uint4*>(op + i * row_stride) = r;
                    }
                }
            }
          }
            __syncwarp();
            if (ok && lane == 0) mbar_arrive(bar(kBarVEmpty + stage));
        }
        // quadrants of the last block that hold no unit: keep the chunk barriers in step
        if (ok && my_blocks > 0 && (my_units & 3) != 0 && qd >= (my_units & 3)) {
            for (int dx = 0; ok && dx < 3; ++dx) {
                const int cs = 3 * (my_blocks - 1) + dx, ds = cs & 1;
                if (!warp_wait(bar(kBarDFull + ds), (cs >> 1) & 1)) { ok = false; break; }
                if (lane == 0) mbar_arrive(bar(kBarDFree + ds));
            }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarVDone));
    } else if (warp == kCtlK || warp == kCtlK2) {
        // =====================================================================================
        // key-side control: the key MMAs (18 per block: 9 taps x two K = 16 halves); warp 16 takes
        // the even blocks, warp 18 the odd ones, in turn.  The tensor pipe executes one small MMA
        // at a time, so the two threads overlap each other's waits rather than their MMAs.
        // =====================================================================================
        uint32_t leader;
        const bool elected = elect_one(leader);
        if (elected && ok) {
            const uint32_t sBk0 = smem_u32(smem + L.bk_off);
            // This thread has one thing to wait for at a time, so it parks in the waits (bounded).
            // The two threads take the blocks in turn: a thread starts block b only when the other
            // one has got past the P-ready wait of the last chunk of block b - 1, so the P-ready
            // barriers are waited on strictly in chunk order.
            const int me = warp == kCtlK ? 0 : 1;
            if (!mbar_wait(bar(kBarWeights), 0)) ok = false;
            for (int blk = me, n = 0; ok && blk < my_blocks; blk += 2, ++n) {
                const int lb = blk & 1;
                const uint32_t dcol = tmem + kColL + 32 * lb;
                // even blocks wait for the odd block before (none before block 0: parity 1 of a
                // fresh barrier tests true), odd blocks for the even block before
                if (!mbar_wait(bar(kBarTurn + me), me == 0 ? (uint32_t)((n - 1) & 1) : (uint32_t)(n & 1))) { ok = false; break; }
                if (!mbar_wait(bar(kBarLFree + lb), ((blk >> 1) & 1) ^ 1)) { ok = false; break; }
#pragma unroll
                for (int dx = 0; dx < 3; ++dx) {
                    const int pc = 3 * blk + dx, pb = pc & 3;
                    UMMA_TL(10, pc);                                       // key MMA thread: before the P-ready wait
                    if (!mbar_wait(bar(kBarPReady + pb), (pc >> 2) & 1)) { ok = false; break; }
                    UMMA_TL(11, pc);
                    if (dx == 2) mbar_arrive(bar(kBarTurn + (me ^ 1)));
                    tc_fence_after_sync();
                    const uint32_t acol = tmem + kColP + 48 * pb;
                    const uint64_t bdesc = umma_smem_desc(sBk0 + (uint32_t)dx * 4u * 512u, 512, 128);
#pragma unroll
                    for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
                        for (int kh = 0; kh < 2; ++kh)      // 16 bytes of descriptor address = 1 unit
                            umma_bf16_ts(dcol, acol + 16 * dy + 8 * kh, bdesc + (uint64_t)((dy * 12 + kh * 2) * 32),
                                         kIdesc32, (dx != 0 || dy != 0 || kh != 0) ? 1u : 0u);
                    }
                    umma_commit(bar(kBarPFree + pb));
                    UMMA_TL(12, pc);                                       // MMAs and commit issued
                    if (dx == 2) umma_commit(bar(kBarLFull + lb));
                }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
        if (warp == kCtlK) {
            if (my_tiles > 0 && !warp_wait(bar(kBarVDone), 0)) ok = false;
            tc_fence_after_sync();
            __syncwarp();
            tmem_dealloc(tmem, kTmemCols);
        }
    } else if (warp == kCtlV) {
        // =====================================================================================
        // value-side control: the value MMAs (chunk c = 3 blk + dx -> TMEM slot c & 1).  One thing to
        // wait for at a time, so the thread parks in the (bounded) waits.
        // =====================================================================================
        uint32_t leader;
        const bool elected = elect_one(leader);
        if (elected && ok) {
            const uint32_t sB0 = smem_u32(smem + L.b_off);
            if (!mbar_wait(bar(kBarWeights), 0)) ok = false;
            for (int blk = 0; ok && blk < my_blocks; ++blk) {
                const int eb = blk & 1;
                if (!mbar_wait(bar(kBarEReady + eb), (blk >> 1) & 1)) { ok = false; break; }
                const uint32_t acol = tmem + kColE + 16 * eb;
#pragma unroll
                for (int dx = 0; dx < 3; ++dx) {
                    const int cs = 3 * blk + dx, ds = cs & 1;
                    UMMA_TL(13, cs);                                       // value MMA thread: before the slot-free wait
                    if (!mbar_wait(bar(kBarDFree + ds), ((cs >> 1) & 1) ^ 1)) { ok = false; break; }
                    UMMA_TL(14, cs);
                    tc_fence_after_sync();
                    const uint32_t sB = sB0 + dx * 12 * 512;
                    const uint32_t idesc = kIdesc96;
                    const uint32_t dcol = tmem + kColD + ds * 112;
                    umma_bf16_ts(dcol, acol, umma_smem_desc(sB, 128, 512), idesc, 0);
                    umma_bf16_ts(dcol, acol + 8, umma_smem_desc(sB + 256, 128, 512), idesc, 1);
                    umma_commit(bar(kBarDFull + ds));
                    UMMA_TL(15, cs);
                    if (dx == 2) umma_commit(bar(kBarEFree + eb));
                }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
    } else {
        // =====================================================================================
        // TMA thread: refills the K/q ring and the V ring as their stages are released
        // =====================================================================================
        uint32_t leader;
        const bool elected = elect_one(leader);
        if (elected && ok) {
            int left = my_tiles - v_issued + my_tiles - k_issued;
            uint32_t idle = 0;
            while (left > 0) {
                const uint32_t tK = mbar_test_u32(bar(kBarKEmpty + kq.stage), (kq.round - 1) & 1);
                const uint32_t tV = mbar_test_u32(bar(kBarVEmpty + vq.stage), (vq.round - 1) & 1);
                const int left_before = left;
                if (tK != 0 && k_issued < my_tiles) { issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; --left; }
                if (tV != 0 && v_issued < my_tiles) {
                    issue_v_tile(vq); walk_next(vq, SV); ++v_issued; --left;
                }
                if (left != left_before) idle = 0;
                else {
                    if (++idle > (1u << 22)) { ok = false; break; }
                    __nanosleep(200);
                }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
    }
    if (!ok && my_tiles > 0 && lane == 0) atomicExch(P.status, 1);
}

}  // namespace

bool umma_ts_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && ksize == 3;
}

namespace {

template <int TW>
cudaError_t setup_one() {
    return cudaFuncSetAttribute(umma_ts_kernel<TW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

// The main kernel is launched with programmatic stream serialisation: it may begin (barrier set-up,
// tensor-memory allocation, first tile loads) while the prep kernel before it in the stream is still
// running; the one thread that reads the prep kernel's output waits for that grid inside the kernel.
template <int TW>
cudaError_t launch_one(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const UmmaParams& P,
                       int grid, cudaStream_t stream) {
    static_assert(v_stages_for(TW) >= 2, "tile width does not fit shared memory");
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_layout(TW, v_stages_for(TW)).total;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, umma_ts_kernel<TW>, mq, mk, mv, P);
}

}  // namespace

size_t umma_ts_workspace_bytes(int heads) { return (size_t)heads * kImgBytes; }

cudaError_t umma_ts_setup() {
    if (!tensor_map_available()) return cudaErrorNotSupported;
    cudaError_t e = setup_one<8>();
    if (e == cudaSuccess) e = setup_one<16>();
    if (e == cudaSuccess) e = setup_one<24>();
    if (e == cudaSuccess) e = setup_one<32>();
    if (e == cudaSuccess) e = setup_one<40>();
    if (e == cudaSuccess) e = setup_one<48>();
    if (e == cudaSuccess) e = setup_one<56>();
    if (e == cudaSuccess) e = setup_one<64>();
    return e;
}

cudaError_t launch_umma_ts_prep(const Problem& p, void* workspace, cudaStream_t stream) {
    umma_ts_prep_kernel<<<dim3((unsigned)p.heads, 6), 256, 0, stream>>>(p.wk, p.wv, static_cast<unsigned char*>(workspace));
    return cudaGetLastError();
}

cudaError_t launch_umma_ts(const Problem& p, const void* workspace, int* d_status, int num_sms, cudaStream_t stream) {
    const int txn = (p.W + 63) / 64;
    const int TW = ((((p.W + txn - 1) / txn) + 7) / 8) * 8;
    UmmaParams P;
    P.bimg = static_cast<const unsigned char*>(workspace); P.bias = p.bias;
    P.out = static_cast<__nv_bfloat16*>(p.out);
    P.status = d_status;
    P.B = p.B; P.H = p.H; P.W = p.W; P.heads = p.heads;
    P.tiles_x = (p.W + TW - 1) / TW;
    P.tiles_y = (p.H + 3) / 4;
    P.scale_log2e = kLog2e / sqrtf((float)kHeadDim);

    const int C = p.heads * kHeadDim;
    CUtensorMap map_q, map_k, map_v;
    if (!make_tile_map(&map_q, p.q, 2, p.B, p.H, p.W, C, kHeadDim, TW, 4) ||
        !make_tile_map(&map_k, p.k, 2, p.B, p.H, p.W, C, kHeadDim, TW + 2, 6) ||
        !make_tile_map(&map_v, p.v, 2, p.B, p.H, p.W, C, kHeadDim, TW + 2, 6))
        return cudaErrorInvalidValue;

    const long long tiles = (long long)P.tiles_x * P.tiles_y * p.B * p.heads;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    int grid = num_sms;
    if (grid < p.heads) grid = p.heads;
    if ((long long)grid > tiles) grid = (int)tiles;
    switch (TW) {
        case 8: return launch_one<8>(map_q, map_k, map_v, P, grid, stream);
        case 16: return launch_one<16>(map_q, map_k, map_v, P, grid, stream);
        case 24: return launch_one<24>(map_q, map_k, map_v, P, grid, stream);
        case 32: return launch_one<32>(map_q, map_k, map_v, P, grid, stream);
        case 40: return launch_one<40>(map_q, map_k, map_v, P, grid, stream);
        case 48: return launch_one<48>(map_q, map_k, map_v, P, grid, stream);
        case 56: return launch_one<56>(map_q, map_k, map_v, P, grid, stream);
        case 64: return launch_one<64>(map_q, map_k, map_v, P, grid, stream);
        default: return cudaErrorInvalidConfiguration;
    }
}

}  // namespace slide_attn

#ifdef SLIDE_ATTN_TIMELINE
// host [16][128]: the clock64 stamps listed at UMMA_TL, indexed by chunk or block; returns the cudaError_t of the copy
extern "C" int slide_attn_umma_ts_timeline(long long* host) {
    return (int)cudaMemcpyFromSymbol(host, slide_attn::g_umma_timeline, sizeof(long long) * 16 * 128);
}
#endif
