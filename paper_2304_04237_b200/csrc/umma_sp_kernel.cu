// UMMA_SP variant (bf16, head_dim 32, k = 3): the arithmetic of UMMA_TS -- both contractions of the
// fused forward on tcgen05.mma with their A operands in tensor memory -- scheduled as ONE team of
// eight compute warps that runs a three-stage software pipeline over the 128-pixel blocks.
//
// Arithmetic (Eq. 2 with Eq. 12 inside; w = E + D, E the one-hot shift of Eq. 11):
//   P[p,(t,c)] = q[p,c] k[p+off(t),c]                          packed bf16 multiply -> tcgen05.st
//   L[p,n]     = sum_{t,c} P[p,(t,c)] Bk[(t,c),n]              key MMA, A from tensor memory
//                n = 0..8: deformed part D_k of slot n;  n = 9..17: plain q.k sum of tap n-9
//   logit[s]   = (L[s] + L[9+s]) scale + bias[s];  e = exp2(logit - max)
//   A' row     = e_hi | e_hi | e_lo | e8_hi e8_hi e8_lo 0..    -> tcgen05.st
//   D[p,(t,c)] = sum_k A'[p,k] Bv[k,(t,c)]  (+16 sum columns)  value MMA, A from tensor memory
//   out[p,c]   = (sum_t D[p,t,c] v[p+off(t),c]) / sum[p]
//
// Schedule.  Warp w of the eight compute warps owns pixel rows 2(w/4), 2(w/4)+1 of the unit (4 rows x
// 8 columns = one TMEM quadrant, w % 4) of every block.  Iteration i of a warp:
//     S(i-1)  wait for the logits of block i-1; the warp whose row pair equals the block's parity
//             does the softmax of its quadrant and stores the A' rows
//     P(i)    q.k products of block i into tensor memory            -> arrive "P ready"
//     V(i-2)  value chunks of block i-2 against the V halo, store   -> arrive "value go"
// and the MMA thread: wait "P ready"(i) -> 18 key MMAs of block i; wait "value go"(i) -> 6 value
// MMAs of block i-1.  Each MMA result is first needed one long phase after its issue, so in steady
// state no wait blocks.  Every region of tensor memory has one writer and one reader per block and
// program order plus these two barriers (and the two commit barriers) order them, so tensor memory
// is single-buffered: P 144 columns, logits 32, A' 2 x 16, value accumulators 304 -- 512 in all.
//
// Every wait is bounded; a wait that runs out sets the status word, and tensor memory is released
// on every path.
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

namespace {

constexpr int kHeadDim = 32;
constexpr int kCWarps = 8;                              // compute warps
constexpr int kWarpMma = kCWarps;                       // warp 8: all MMAs, owns tensor memory
constexpr int kWarpTma = kCWarps + 1;                   // warp 9: TMA thread, K/q and V tiles
constexpr int kThreads = (kWarpTma + 1) * 32;
constexpr int kKStages = 2;
constexpr int kMaxVStages = 3;
constexpr int kBCols = 304;                             // 288 value columns + 16 sum columns
constexpr int kBBytes = kBCols * 64;
constexpr int kBkBytes = 36 * 512;                      // key-side B: 288 K x 32 N bf16
constexpr int kWeightBytes = kHeadDim * 81 * 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kTmemCols = 512;
// tensor-memory columns
constexpr uint32_t kColP = 0;                           // q.k products of one block: 9 taps x 16 columns
constexpr uint32_t kColL = 144;                         // logit tile, 32 columns
constexpr uint32_t kColE = 176;                         // two A' tiles of 16 columns (block parity)
constexpr uint32_t kColD = 208;                         // value accumulators: 3 chunks of 96 (+16 sum columns)
constexpr uint32_t kIdesc96 = umma_idesc_bf16(128, 96);
constexpr uint32_t kIdesc112 = umma_idesc_bf16(128, 112);
constexpr uint32_t kIdesc32 = umma_idesc_bf16(128, 32);

struct SpParams {
    const float* wk;
    const float* wv;
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
    const uint32_t wbytes = ((uint32_t)(2 * kWeightBytes) + 1023u) & ~1023u;
    if (s.halo_pad < wbytes) s.halo_pad = wbytes;
    s.kstage_bytes = s.halo_pad + (((uint32_t)(4 * TW * 64) + 1023u) & ~1023u);
    s.v_off = kKStages * s.kstage_bytes;
    s.b_off = s.v_off + vstages * s.halo_pad;
    s.bk_off = s.b_off + kBBytes;
    s.tmem_off = s.bk_off + kBkBytes;
    s.bar_off = s.tmem_off + 16;
    s.total = s.bar_off + 24 * 8 + 1024;
    return s;
}

constexpr size_t kMaxSmem = 227 * 1024;

__host__ __device__ constexpr int v_stages_for(int TW) {
    for (int st = kMaxVStages; st >= 2; --st)
        if (smem_layout(TW, st).total <= kMaxSmem) return st;
    return 0;
}

constexpr int kBarKFull = 0;         // [2]
constexpr int kBarKEmpty = 2;        // [2]  count 8
constexpr int kBarVFull = 4;         // [3]
constexpr int kBarVEmpty = 7;        // [3]  count 8
constexpr int kBarWeights = 10;
constexpr int kBarWeightsDone = 11;  // count 10 (every warp)
constexpr int kBarPReady = 12;       // count 8: P of a block stored          (phase = block)
constexpr int kBarLFull = 13;        // key MMAs of a block complete          (phase = block)
constexpr int kBarValGo = 14;        // count 8: A' stored and D read         (phase = block of the A')
constexpr int kBarDFull = 15;        // [3] value chunk complete              (phase = block)
constexpr int kBarDone = 18;         // count 8

__device__ __forceinline__ uint4 lds_u4(const unsigned char* base, uint32_t off) {
    return *reinterpret_cast<const uint4*>(base + off);
}
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}

template <int TW>
__global__ void __launch_bounds__(kThreads, 1)
umma_sp_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const SpParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int SV = v_stages_for(TW);
    constexpr Smem L = smem_layout(TW, SV);
    const uint32_t bar0 = smem_u32(smem + L.bar_off);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3;
    constexpr int U = TW >> 3;
    constexpr int HW2 = TW + 2;

    const int h = blockIdx.x % P.heads;
    const int rank = blockIdx.x / P.heads;
    const int nrank = ((int)gridDim.x - h + P.heads - 1) / P.heads;
    const int tiles_per_head = P.B * P.tiles_y * P.tiles_x;
    const int my_tiles = rank < tiles_per_head ? (tiles_per_head - rank + nrank - 1) / nrank : 0;
    const int my_units = my_tiles * U;
    const int nb = (my_units + 3) >> 2;
    const int C = P.heads * kHeadDim;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kKStages; ++s) { mbar_init(bar(kBarKFull + s), 1); mbar_init(bar(kBarKEmpty + s), kCWarps); }
        for (int s = 0; s < kMaxVStages; ++s) { mbar_init(bar(kBarVFull + s), 1); mbar_init(bar(kBarVEmpty + s), kCWarps); }
        mbar_init(bar(kBarWeights), 1);
        mbar_init(bar(kBarWeightsDone), kThreads / 32);
        mbar_init(bar(kBarPReady), kCWarps);
        mbar_init(bar(kBarLFull), 1);
        mbar_init(bar(kBarValGo), kCWarps);
        for (int i = 0; i < 3; ++i) mbar_init(bar(kBarDFull + i), 1);
        mbar_init(bar(kBarDone), kCWarps);
    }
    if (warp == kWarpMma) tmem_alloc(smem_u32(smem + L.tmem_off), kTmemCols);
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

    // weights are staged in the last V stage; the weights, the first K/q tiles and the first V tiles
    // are sent for at once
    const unsigned char* w_stage = smem + L.v_off + (size_t)(SV - 1) * L.halo_pad;
    int k_issued = 0, v_issued = 0;
    TileWalk kq = walk_begin(), vq = kq;
    if (my_tiles > 0 && warp == kWarpMma && lane == 0) {
        mbar_expect_tx(bar(kBarWeights), 2 * kWeightBytes);
        bulk_load_1d(smem_u32(w_stage), P.wk + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
        bulk_load_1d(smem_u32(w_stage) + kWeightBytes, P.wv + (size_t)h * kHeadDim * 81, kWeightBytes, bar(kBarWeights));
    }
    if (my_tiles > 0 && warp == kWarpTma) {
        // the same lane is elected here and in the refill loop below (the election is deterministic for
        // a given member mask), so the ring positions it advances here are the ones it continues from
        uint32_t leader;
        if (elect_one(leader)) {
            while (k_issued < my_tiles && k_issued < kKStages) { issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; }
            while (v_issued < my_tiles && v_issued < SV - 1) { issue_v_tile(vq); walk_next(vq, SV); ++v_issued; }
        }
    }
    __syncwarp();

    bool ok = my_tiles > 0 && warp_wait(bar(kBarWeights), 0);
    const float* wks = reinterpret_cast<const float*>(w_stage);
    const float* wvs = wks + kHeadDim * 81;

    if (ok) {
        // ---- value-side B tile: column n = (tap-column-major tap, channel), 64 bytes of K each --------
        unsigned char* sB = smem + L.b_off;
        for (int n = threadIdx.x; n < kBCols; n += kThreads) {
            unsigned char* col = sB + (n >> 3) * 512 + (n & 7) * 16;
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) w[i] = 0u;
            if (n >= 288) {
#pragma unroll
                for (int i = 4; i < 12; ++i) w[i] = kOnesBf16x2;
                w[12] = pack_bf16(0.f, 1.f); w[13] = pack_bf16(1.f, 0.f);
            } else {
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
        }
        // ---- key-side B: [k-group of 8][n-group of 8][8 n rows][8 k] bf16; K index = 32 tap + kappa,
        // kappa -> channel as the product phase's tcgen05.st lays P out
        unsigned char* sBk = smem + L.bk_off;
        for (int item = threadIdx.x; item < 36 * 32; item += kThreads) {
            const int n = item & 31, kg = item >> 5;
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
        fence_proxy_async_smem();
    }
    __syncthreads();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(kBarWeightsDone));

    if (warp < kCWarps) {
        // =====================================================================================
        // compute warps
        // =====================================================================================
        const int q = warp & 3;                                    // TMEM quadrant = unit of the block
        const int pm = warp >> 2;                                  // pixel-row pair of the unit
        const uint32_t tq = tmem + ((uint32_t)(32 * q) << 16);     // the quadrant (softmax: thread = lane)
        const uint32_t th = tmem + ((uint32_t)(32 * q + 16 * pm) << 16);   // this warp's 16 lanes
        float biasl[9];
#pragma unroll
        for (int s = 0; s < 9; ++s) biasl[s] = P.bias ? P.bias[h * 9 + s] * kLog2e : 0.f;

        // tile rings: every warp visits every tile of each ring in order (waits for it, releases it
        // once), so that arrivals always land in the phase they belong to; a tile is released as soon
        // as the warp's next unit lies beyond it
        int k_cur = -1, v_cur = -1;
        bool k_rel = false, v_rel = false;
        TileWalk vw = walk_begin();                                // coordinates of tile v_cur
        auto k_release = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarKEmpty + k_cur % kKStages));
            k_rel = true;
        };
        auto v_release = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarVEmpty + v_cur % SV));
            v_rel = true;
        };
        auto k_advance = [&](int ti) -> bool {
            while (k_cur < ti) {
                if (k_cur >= 0 && !k_rel) k_release();
                ++k_cur; k_rel = false;
                if (!warp_wait(bar(kBarKFull + k_cur % kKStages), (uint32_t)(k_cur / kKStages) & 1u)) return false;
            }
            return true;
        };
        auto v_advance = [&](int ti) -> bool {
            while (v_cur < ti) {
                if (v_cur >= 0) { if (!v_rel) v_release(); walk_next(vw, SV); }
                ++v_cur; v_rel = false;
                if (!warp_wait(bar(kBarVFull + v_cur % SV), (uint32_t)(v_cur / SV) & 1u)) return false;
            }
            return true;
        };

        for (int i = 0; ok && i < nb + 2; ++i) {
            // ---------------- S(i-1): logits of block i-1 -> A' rows ----------------
            if (i >= 1 && i - 1 < nb) {
                const int sb = i - 1;
                if (!warp_wait(bar(kBarLFull), (uint32_t)sb & 1u)) { ok = false; break; }
                if (pm == (sb & 1) && 4 * sb + q < my_units) {
                    tc_fence_after_sync();
                    float Lg[32];
                    tmem_ld_32x32b_x32(tq + kColL, Lg);
                    uint32_t row[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) row[j] = 0u;
                    float l[9], m = -INFINITY;
#pragma unroll
                    for (int s = 0; s < 9; ++s) { l[s] = (Lg[s] + Lg[9 + s]) * P.scale_log2e + biasl[s]; m = fmaxf(m, l[s]); }
                    float hi[9], lo[9];
#pragma unroll
                    for (int s = 0; s < 9; ++s) {
                        const float e = fast_exp2(l[s] - m);
                        hi[s] = __bfloat162float(__float2bfloat16_rn(e));
                        lo[s] = e - hi[s];
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        row[j] = pack_bf16(hi[2 * j], hi[2 * j + 1]);
                        row[4 + j] = row[j];
                        row[8 + j] = pack_bf16(lo[2 * j], lo[2 * j + 1]);
                    }
                    row[12] = pack_bf16(hi[8], hi[8]);
                    row[13] = pack_bf16(lo[8], 0.f);
                    tmem_st_32x32b_x16(tq + kColE + 16 * (sb & 1), row);
                    tmem_wait_st();
                }
            }
            // ---------------- P(i): q.k products of block i ----------------
            if (i < nb) {
                const int u = 4 * i + q;
                const bool valid = u < my_units;
                // a warp without a unit here still visits the tiles it passes
                const int ti = valid ? u / U : my_tiles - 1;
                if (!k_advance(ti)) { ok = false; break; }
                if (valid) {
                    const int ul = u - ti * U, ux = ul * 8;
                    const unsigned char* sK = smem + (size_t)(ti % kKStages) * L.kstage_bytes;
                    const unsigned char* sQ = sK + L.halo_pad;
                    uint32_t qf[2][4];                             // pixel rows 2pm, 2pm+1 of column ux + g
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const uint4 v = lds_u4(sQ, (uint32_t)((2 * pm + r) * TW + ux + g) * 64u + tig * 16u);
                        qf[r][0] = v.x; qf[r][1] = v.y; qf[r][2] = v.z; qf[r][3] = v.w;
                    }
                    const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;
                    tc_fence_after_sync();
#pragma unroll
                    for (int dx = 0; dx < 3; ++dx) {
                        uint4 kc[4];                               // halo rows 2pm .. 2pm+3 of column dx
#pragma unroll
                        for (int r = 0; r < 4; ++r) kc[r] = lds_u4(sK, off0 + (uint32_t)((2 * pm + r) * HW2 + dx) * 64u);
#pragma unroll
                        for (int dy = 0; dy < 3; ++dy) {
                            const uint4 k0 = kc[dy], k1 = kc[dy + 1];
                            uint32_t r[8];
                            r[0] = hmul2_bf16(qf[0][0], k0.x); r[1] = hmul2_bf16(qf[0][1], k0.y);
                            r[2] = hmul2_bf16(qf[1][0], k1.x); r[3] = hmul2_bf16(qf[1][1], k1.y);
                            r[4] = hmul2_bf16(qf[0][2], k0.z); r[5] = hmul2_bf16(qf[0][3], k0.w);
                            r[6] = hmul2_bf16(qf[1][2], k1.z); r[7] = hmul2_bf16(qf[1][3], k1.w);
                            tmem_st_16x256b_x2(th + kColP + 16 * (3 * dy + dx), r);
                        }
                    }
                    tmem_wait_st();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPReady));
                {   // tiles strictly before the next unit's tile are visited and released now
                    const int nti = u + 4 < my_units ? (u + 4) / U : my_tiles;
                    if (!k_advance(nti - 1)) { ok = false; break; }
                    if (!k_rel && nti > k_cur) k_release();
                }
            }
            // ---------------- V(i-2): value chunks of block i-2 ----------------
            if (i >= 2) {
                const int vb = i - 2;
                const int u = 4 * vb + q;
                const bool valid = u < my_units;
                const int ti = valid ? u / U : my_tiles - 1;
                const int ux = valid ? (u - ti * U) * 8 : 0;
                if (!v_advance(ti)) { ok = false; break; }
                const unsigned char* sV = smem + L.v_off + (size_t)(ti % SV) * L.halo_pad;
                const uint32_t off0 = (uint32_t)(ux + g) * 64u + tig * 16u;
                uint4 vp[3][4];
                if (valid) {
#pragma unroll
                    for (int dx = 0; dx < 3; ++dx)
#pragma unroll
                        for (int r = 0; r < 4; ++r) vp[dx][r] = lds_u4(sV, off0 + (uint32_t)((2 * pm + r) * HW2 + dx) * 64u);
                }
                float o_acc[2][8];
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int c = 0; c < 8; ++c) o_acc[r][c] = 0.f;
                float inv[2] = {0.f, 0.f};
#pragma unroll
                for (int dx = 0; dx < 3; ++dx) {
                    if (!warp_wait(bar(kBarDFull + dx), (uint32_t)vb & 1u)) { ok = false; break; }
                    if (valid) {
                        tc_fence_after_sync();
                        uint32_t dr[48];
                        const uint32_t ta = th + kColD + 96 * dx;
                        tmem_ld3_16x256b_x4_nowait(ta, ta + 32, ta + 64, dr);
                        uint32_t sr[4] = {0u, 0u, 0u, 0u};         // sum_s e[p,s] of the two pixels (last chunk)
                        if (dx == 2) tmem_ld_16x256b_x1_nowait(th + kColD + 288, sr);
                        float vf[4][8];
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const uint4 v = vp[dx][r];
                            vf[r][0] = bf16_lo(v.x); vf[r][1] = bf16_hi(v.x);
                            vf[r][2] = bf16_lo(v.y); vf[r][3] = bf16_hi(v.y);
                            vf[r][4] = bf16_lo(v.z); vf[r][5] = bf16_hi(v.z);
                            vf[r][6] = bf16_lo(v.w); vf[r][7] = bf16_hi(v.w);
                        }
                        tmem_wait_ld48(dr);
                        if (dx == 2) {
                            tmem_pass4(sr);
                            inv[0] = rcp_approx(__uint_as_float(sr[0])); inv[1] = rcp_approx(__uint_as_float(sr[2]));
                        }
                        float d[48];
#pragma unroll
                        for (int j = 0; j < 48; ++j) d[j] = __uint_as_float(dr[j]);
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
                }
                if (!ok) break;
                if (valid) {
                    const int x = vw.tx * TW + ux + g, y0 = vw.ty * 4 + 2 * pm;
                    __nv_bfloat16* op = P.out + ((size_t)(vw.b * P.H + y0) * P.W + x) * C + h * kHeadDim + tig * 8;
                    const size_t row_stride = (size_t)P.W * C;
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        if (x < P.W && y0 + r < P.H) {
                            uint4 o;
                            o.x = pack_bf16(o_acc[r][0] * inv[r], o_acc[r][1] * inv[r]);
                            o.y = pack_bf16(o_acc[r][2] * inv[r], o_acc[r][3] * inv[r]);
                            o.z = pack_bf16(o_acc[r][4] * inv[r], o_acc[r][5] * inv[r]);
                            o.w = pack_bf16(o_acc[r][6] * inv[r], o_acc[r][7] * inv[r]);
                            *reinterpret_cast<uint4*>(op + r * row_stride) = o;
                        }
                    }
                }
                {
                    const int nti = u + 4 < my_units ? (u + 4) / U : my_tiles;
                    if (!v_advance(nti - 1)) { ok = false; break; }
                    if (!v_rel && nti > v_cur) v_release();
                }
            }
            // the A' rows of block i-1 are stored and the accumulators of block i-2 are read: the value
            // MMAs of block i-1 may go
            if (i >= 1 && i <= nb) {
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarValGo));
            }
        }
        // visit what is left of the two tile rings, so that no copy is in flight when the CTA ends
        if (ok && !k_advance(my_tiles - 1)) ok = false;
        if (ok && !v_advance(my_tiles - 1)) ok = false;
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarDone));
    } else if (warp == kWarpMma) {
        // =====================================================================================
        // MMA thread: key MMAs of block j after "P ready"(j), value MMAs of block j-1 after "value go"(j)
        // =====================================================================================
        uint32_t leader;
        const bool elected = elect_one(leader);
        if (elected && ok) {
            const uint32_t sBk0 = smem_u32(smem + L.bk_off);
            const uint32_t sB0 = smem_u32(smem + L.b_off);
            for (int j = 0; ok && j <= nb; ++j) {
                if (j < nb) {
                    if (!mbar_wait(bar(kBarPReady), (uint32_t)j & 1u)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t dcol = tmem + kColL;
#pragma unroll
                    for (int t = 0; t < 9; ++t) {
#pragma unroll
                        for (int kh = 0; kh < 2; ++kh)
                            umma_bf16_ts(dcol, tmem + kColP + 16 * t + 8 * kh,
                                         umma_smem_desc(sBk0 + (uint32_t)(4 * t + 2 * kh) * 512u, 512, 128), kIdesc32,
                                         (t != 0 || kh != 0) ? 1u : 0u);
                    }
                    umma_commit(bar(kBarLFull));
                }
                if (j >= 1) {
                    const int vb = j - 1;
                    if (!mbar_wait(bar(kBarValGo), (uint32_t)vb & 1u)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t acol = tmem + kColE + 16 * (vb & 1);
#pragma unroll
                    for (int dx = 0; dx < 3; ++dx) {
                        const uint32_t sB = sB0 + dx * 12 * 512;
                        const uint32_t idesc = dx == 2 ? kIdesc112 : kIdesc96;
                        const uint32_t dcol = tmem + kColD + 96 * dx;
                        umma_bf16_ts(dcol, acol, umma_smem_desc(sB, 128, 512), idesc, 0);
                        umma_bf16_ts(dcol, acol + 8, umma_smem_desc(sB + 256, 128, 512), idesc, 1);
                        umma_commit(bar(kBarDFull + dx));
                    }
                }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
        if (my_tiles > 0 && !warp_wait(bar(kBarDone), 0)) ok = false;
        tc_fence_after_sync();
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    } else {
        // =====================================================================================
        // TMA thread: refills the K/q ring and the V ring as their stages are released
        // =====================================================================================
        uint32_t leader;
        const bool elected = elect_one(leader);
        if (elected && ok) {
            bool weights_done = false;
            int left = my_tiles - v_issued + my_tiles - k_issued;
            uint32_t idle = 0;
            while (left > 0) {
                if (!weights_done) weights_done = mbar_test(bar(kBarWeightsDone), 0);
                const uint32_t tK = mbar_test_u32(bar(kBarKEmpty + kq.stage), (kq.round - 1) & 1);
                const uint32_t tV = mbar_test_u32(bar(kBarVEmpty + vq.stage), (vq.round - 1) & 1);
                const int left_before = left;
                if (tK != 0 && k_issued < my_tiles) { issue_k_tile(kq); walk_next(kq, kKStages); ++k_issued; --left; }
                // the last V stage held the weights: its first tile waits until every warp is done with them
                if (tV != 0 && v_issued < my_tiles && (v_issued != SV - 1 || weights_done)) {
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

template <int TW>
cudaError_t setup_one() {
    return cudaFuncSetAttribute(umma_sp_kernel<TW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

template <int TW>
cudaError_t launch_one(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const SpParams& P,
                       int grid, cudaStream_t stream) {
    static_assert(v_stages_for(TW) >= 2, "tile width does not fit shared memory");
    umma_sp_kernel<TW><<<grid, kThreads, smem_layout(TW, v_stages_for(TW)).total, stream>>>(mq, mk, mv, P);
    return cudaGetLastError();
}

}  // namespace

bool umma_sp_supports(slide_attn_dtype dtype, int head_dim, int ksize) {
    return dtype == SLIDE_ATTN_BF16 && head_dim == kHeadDim && ksize == 3;
}

cudaError_t umma_sp_setup() {
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

cudaError_t launch_umma_sp(const Problem& p, int* d_status, int num_sms, cudaStream_t stream) {
    const int txn = (p.W + 63) / 64;
    const int TW = ((((p.W + txn - 1) / txn) + 7) / 8) * 8;
    SpParams P;
    P.wk = p.wk; P.wv = p.wv; P.bias = p.bias;
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
