// Projections of a Slide-Attention block (Eq. 1: q = x W_q, k = x W_k, v = x W_v; Eq. 3: Concat(heads) W_o)
// as one persistent tcgen05 GEMM:  Y[rows x N] = X[rows x K] W[K x N], X and Y bf16 (token-major, channels
// contiguous), W given in fp32 and rounded to bf16 once as each CTA lays it out in its shared memory, fp32
// accumulation in tensor memory.  One launch per projection call (several when the weights of all output columns
// do not fit shared memory together).
//
// The column range of one launch is split into chunks of `nch` columns (one MMA shape); all chunk images of the
// launch stay resident in shared memory, X comes in as 128-row tiles through a TMA ring.  K <= 256 is one tile
// deep, so a work item (row tile, chunk) is K/16 MMAs of M = 128, N = nch, followed by one commit.
//
// Shared-memory operand layout (no swizzle, K-major core matrices of 8 rows x 16 bytes):
//   X tile   [K/8][128 rows][16 B]   written by K/8 TMA boxes of 8 channels x 128 rows (rows past the end read 0)
//   W chunk  [K/8][nch cols][16 B]   built from the fp32 weights by the epilogue warps while the first X tiles load
// The X boxes fetch a 32-byte sector for every 16 bytes, and with the three output tensors that L2 traffic is what
// bounds the kernel.  Measured and not kept: four producer warps copying the tile with cp.async in row-major order
// of the source (whole lines; planes padded by 16 bytes against bank conflicts; one or two free stages beyond the
// tiles in flight) - 32.5 / 18.0 us for the two projections of a 64-channel block against 21.1 / 12.7 with the boxes.
//
// Warps: 0 TMA producer, 1 MMA issuer (owns tensor memory), 2-17 epilogue in four groups of four (TMEM lane quarter
// = warp % 4; a group owns every fourth work item, because one item's epilogue is a chain of dependent latencies of
// about 850 cycles: one thread per accumulator row, tcgen05.ld.32x32b -> bf16 -> a padded staging patch in shared
// memory -> row-major 16-byte stores of whole sectors).  Tensor memory holds 512 / nch accumulator slots (at most
// eight), so the MMAs run ahead of the epilogue.  Every wait is bounded; a wait that runs out sets the
// status word and the kernel still releases tensor memory.
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

// Time-line build (-DSLIDE_ATTN_TIMELINE, `python -m paper_2304_04237_b200.build --timeline`): CTA 0 stamps clock64
// at six points of its role loops, per work item; slide_attn_proj_timeline copies the stamps out.  The stamps cost a
// few instructions and skip no work; the library proper is built without them.
#ifdef SLIDE_ATTN_TIMELINE
__device__ long long g_proj_timeline[6][256];
#define PROJ_TL(role, idx) do { if (blockIdx.x == 0 && (idx) < 256) g_proj_timeline[role][idx] = clock64(); } while (0)
#else
#define PROJ_TL(role, idx) do {} while (0)
#endif

namespace {

constexpr int kGroups = 4;                   // epilogue warp groups; group g owns the items it = g (mod kGroups)
constexpr int kEpiWarps = 4 * kGroups;       // one warp per TMEM lane quarter in every group
constexpr int kThreads = (2 + kEpiWarps) * 32;
constexpr int kMaxStages = 6;
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxSlots = 8;                 // accumulator slots in tensor memory: 512 / nch, at most this many
constexpr size_t kMaxSmem = 227 * 1024;

constexpr int kBarXFull = 0;                 // [kMaxStages]
constexpr int kBarXEmpty = kMaxStages;       // [kMaxStages]  one arrival: the commit behind the tile's last MMA
constexpr int kBarWeights = 2 * kMaxStages;  // count kEpiWarps: the weight images are in shared memory
constexpr int kBarAccFull = kBarWeights + 1; // [kMaxSlots]
constexpr int kBarAccFree = kBarAccFull + kMaxSlots; // [kMaxSlots]  count 4: the four warps of the group that owned the item
constexpr int kNumBars = kBarAccFree + kMaxSlots;

struct ProjParams {
    const float* w;              // nmat row-major [K][ycols] matrices, one after the other
    __nv_bfloat16* y[3];         // output tensors, each [rows][ycols]
    int ycols;                   // channels of one output tensor = columns of one weight matrix
    int n0;                      // first column of this launch, counted over the concatenated output tensors
    int rows, K, nch, nchunks, stages;
    int sw_max;                  // widest epilogue pass in columns: 64 or 32 (sizes the staging patches)
    int* status;
};


// One epilogue pass of a warp: SW accumulator columns of its 32 rows -> bf16 -> global memory (see the kernel).
template <int SW>
__device__ __forceinline__ void store_cols(uint32_t taddr, unsigned char* stg, int lane, __nv_bfloat16* ybase, int ycols,
                                           int rows_left)
{
    constexpr int RS = SW * 2 + 16;
    uint32_t r[SW];
    // all loads of the pass are in flight before the one wait
#pragma unroll
    for (int c = 0; c < SW; c += 16)
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(r[c + 0]), "=r"(r[c + 1]), "=r"(r[c + 2]), "=r"(r[c + 3]), "=r"(r[c + 4]), "=r"(r[c + 5]), "=r"(r[c + 6]),
              "=r"(r[c + 7]), "=r"(r[c + 8]), "=r"(r[c + 9]), "=r"(r[c + 10]), "=r"(r[c + 11]), "=r"(r[c + 12]), "=r"(r[c + 13]),
              "=r"(r[c + 14]), "=r"(r[c + 15])
            : "r"(taddr + (uint32_t)c) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int c = 0; c < SW; c += 8) {
        // the registers are passed through an empty asm so that no use of them is scheduled above the wait
        asm volatile("" : "+r"(r[c]), "+r"(r[c + 1]), "+r"(r[c + 2]), "+r"(r[c + 3]), "+r"(r[c + 4]), "+r"(r[c + 5]), "+r"(r[c + 6]), "+r"(r[c + 7]));
        *reinterpret_cast<uint4*>(stg + lane * RS + c * 2) =
            make_uint4(pack_bf16(__uint_as_float(r[c]), __uint_as_float(r[c + 1])), pack_bf16(__uint_as_float(r[c + 2]), __uint_as_float(r[c + 3])),
                       pack_bf16(__uint_as_float(r[c + 4]), __uint_as_float(r[c + 5])), pack_bf16(__uint_as_float(r[c + 6]), __uint_as_float(r[c + 7])));
    }
    __syncwarp();
    constexpr int PR = SW / 8;                            // 16-byte pieces per row
    uint4 piece[PR];
#pragma unroll
    for (int j = 0; j < PR; ++j) {
        const int p = j * 32 + lane;
        piece[j] = *reinterpret_cast<const uint4*>(stg + (p / PR) * RS + (p % PR) * 16);
    }
#pragma unroll
    for (int j = 0; j < PR; ++j) {
        const int p = j * 32 + lane, rr = p / PR, pc = p % PR;
        if (rr < rows_left) *reinterpret_cast<uint4*>(ybase + (size_t)rr * ycols + pc * 8) = piece[j];
    }
    __syncwarp();
}

__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}

__global__ void __launch_bounds__(kThreads, 1)
proj_kernel(const __grid_constant__ CUtensorMap map_x, const ProjParams P)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    const uint32_t img_bytes = (uint32_t)P.nchunks * (uint32_t)(P.K >> 3) * (uint32_t)P.nch * 16u;
    const uint32_t img_pad = (img_bytes + 127u) & ~127u;
    const uint32_t stage_bytes = (uint32_t)P.K * 256u;
    const uint32_t x_off = img_pad;
    const uint32_t tmem_off = x_off + (uint32_t)P.stages * stage_bytes;
    const uint32_t bar0 = smem_u32(smem + tmem_off + 16);
    const uint32_t stage_off = (tmem_off + 16 + 16 + kNumBars * 8 + 15u) & ~15u;   // epilogue staging, 16-byte aligned
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int ntiles = (P.rows + 127) >> 7;
    const int my_tiles = (int)blockIdx.x < ntiles ? (ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int S = P.stages;
    const int nslots = 512 / P.nch < kMaxSlots ? 512 / P.nch : kMaxSlots;      // >= 2: nch <= 256

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init_only(bar(kBarXFull + s), 1); mbar_init_only(bar(kBarXEmpty + s), 1); }
        mbar_init_only(bar(kBarWeights), kEpiWarps);
        for (int i = 0; i < kMaxSlots; ++i) { mbar_init_only(bar(kBarAccFull + i), 1); mbar_init_only(bar(kBarAccFree + i), 4); }
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(smem + tmem_off), kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<const volatile uint32_t*>(smem + tmem_off);
    bool ok = true;

    if (warp == 0) {
        // ---- TMA producer: the X tiles of this CTA through the ring.  The kernel may have been launched before the
        // kernels ahead of it in the stream completed, so every thread that reads global memory waits for them first.
        uint32_t leader;
        if (elect_one(leader) && my_tiles > 0) {
            grid_dependency_wait();
            int s = 0, phase = 0;                                // stage t % S and the parity of its t / S-th use
            for (int t = 0, m = (int)blockIdx.x; ok && t < my_tiles; ++t, m += (int)gridDim.x) {
                if (!mbar_wait(bar(kBarXEmpty + s), (uint32_t)(phase ^ 1))) { ok = false; break; }
                const uint32_t dst = smem_u32(smem + x_off + (size_t)s * stage_bytes), fb = bar(kBarXFull + s);
                mbar_expect_tx(fb, stage_bytes);
                for (int kg = 0; kg < (P.K >> 3); ++kg) tma_load_4d(dst + (uint32_t)kg * 2048u, &map_x, fb, 8 * kg, m * 128, 0, 0);
                if (++s == S) { s = 0; phase ^= 1; }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
    } else if (warp == 1) {
        // ---- MMA issuer
        uint32_t leader;
        if (elect_one(leader) && my_tiles > 0) {
            const uint32_t idesc = umma_idesc_bf16(128, (uint32_t)P.nch);
            const uint32_t chunk_bytes = (uint32_t)(P.K >> 3) * (uint32_t)P.nch * 16u;
            const uint32_t b_lbo = (uint32_t)P.nch * 16u;
            const uint32_t sB0 = smem_u32(smem);
            if (!mbar_wait(bar(kBarWeights), 0)) ok = false;
            int s = 0, phase = 0, slot = 0, slot_phase = 0, it = 0;
            for (int t = 0; ok && t < my_tiles; ++t) {
                if (!mbar_wait(bar(kBarXFull + s), (uint32_t)phase)) { ok = false; break; }
                // descriptors step in 16-byte units: two planes of X and two K-groups of the chunk per MMA
                const uint64_t adesc0 = umma_smem_desc(smem_u32(smem + x_off + (size_t)s * stage_bytes), 2048, 128);
                uint64_t bdesc0 = umma_smem_desc(sB0, b_lbo, 128);
                for (int ch = 0; ch < P.nchunks; ++ch, ++it, bdesc0 += chunk_bytes >> 4) {
                    PROJ_TL(0, it);                              // MMA thread turns to the item
                    if (!mbar_wait(bar(kBarAccFree + slot), (uint32_t)(slot_phase ^ 1))) { ok = false; break; }
                    PROJ_TL(1, it);                              // its accumulator slot is free
                    tc_fence_after_sync();
                    const uint32_t dcol = tmem + (uint32_t)(slot * P.nch);
                    uint64_t adesc = adesc0, bdesc = bdesc0;
                    for (int kk = 0; kk < (P.K >> 4); ++kk, adesc += 4096u >> 4, bdesc += (2u * b_lbo) >> 4)
                        umma_bf16_ss(dcol, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
                    umma_commit(bar(kBarAccFull + slot));
                    PROJ_TL(2, it);                              // MMAs and commit issued
                    if (++slot == nslots) { slot = 0; slot_phase ^= 1; }
                }
                if (ok) umma_commit(bar(kBarXEmpty + s));       // the tile's last MMA has read it
                if (++s == S) { s = 0; phase ^= 1; }
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
    } else {
        // ---- epilogue: lane = accumulator row 32 (warp % 4) + lane of the tile.  Each pass takes up to 64 columns:
        // the lane's row goes TMEM -> registers -> bf16 -> a staging row of this warp in shared memory (row pitch
        // 2 SW + 16 bytes: conflict-free 16-byte stores), then the warp writes the 32 x SW patch to global memory in
        // row-major order, 16 bytes per lane, so that every row segment leaves as whole 32-byte sectors.
        const int sub = warp & 3, group = (warp - 2) >> 2;
        const uint32_t tlane = tmem + ((uint32_t)(32 * sub) << 16);
        unsigned char* stg = smem + stage_off + (size_t)(warp - 2) * (size_t)(32 * (P.sw_max * 2 + 16));
        if (my_tiles > 0) {
            // the bf16 weight images of this launch's columns: [chunk][K/8][nch][8 K-consecutive bf16]; consecutive
            // threads take consecutive columns, so the fp32 reads are coalesced
            grid_dependency_wait();
            const int ncl = P.nchunks * P.nch, kgs = P.K >> 3;
            const uint32_t chunk_bytes = (uint32_t)kgs * (uint32_t)P.nch * 16u;
            for (int item = (int)threadIdx.x - 64; item < kgs * ncl; item += kEpiWarps * 32) {
                const int kg = item / ncl, nl = item - kg * ncl;
                const int n = P.n0 + nl, mat = n / P.ycols, col = n - mat * P.ycols;
                const float* src = P.w + ((size_t)mat * P.K + 8 * kg) * P.ycols + col;
                float val[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) val[e] = src[(size_t)e * P.ycols];
                const int chn = nl / P.nch;
                *reinterpret_cast<uint4*>(smem + (size_t)chn * chunk_bytes + ((size_t)kg * P.nch + (nl - chn * P.nch)) * 16) =
                    make_uint4(pack_bf16(val[0], val[1]), pack_bf16(val[2], val[3]), pack_bf16(val[4], val[5]), pack_bf16(val[6], val[7]));
            }
            fence_proxy_async_smem();            // the tensor core reads these bytes through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarWeights));
        }
        // items in launch order: it = t * nchunks + ch.  This warp's group owns the items it = group (mod ngroups): it
        // waits for, reads and releases only those; for the others it merely advances the slot and column counters.
        // No more groups take part than there are slots: a group then always waits on a phase of a slot's barrier whose
        // predecessor it knows to be complete (its previous item came later than this slot's previous use), so the
        // parity test cannot be satisfied by an older phase.
        const int ngroups = nslots < kGroups ? nslots : kGroups;
        const int t0 = P.n0 / P.ycols, c00 = P.n0 - t0 * P.ycols;     // tensor and column of the launch's first chunk
        int slot = 0, slot_phase = 0, turn = 0, it = 0;               // turn = it mod ngroups
        for (int t = 0; ok && t < my_tiles; ++t) {
            const long long row0 = ((long long)blockIdx.x + (long long)t * gridDim.x) * 128 + 32 * sub;
            const int rows_left = (long long)P.rows - row0 > 32 ? 32 : (int)((long long)P.rows - row0);   // may be <= 0
            int ti = t0, col0 = c00;                                  // a chunk lies within one tensor
            for (int ch = 0; ch < P.nchunks; ++ch, ++it) {
                if (turn == group) {
                    if (sub == 0 && lane == 0) PROJ_TL(3, it);   // the owning group's first warp turns to the item
                    if (!warp_wait(bar(kBarAccFull + slot), (uint32_t)slot_phase)) { ok = false; break; }
                    if (sub == 0 && lane == 0) PROJ_TL(4, it);   // accumulator seen
                    tc_fence_after_sync();
                    const uint32_t tacc = tlane + (uint32_t)(slot * P.nch);
                    __nv_bfloat16* ybase = P.y[ti] + (size_t)row0 * P.ycols + col0;
                    for (int c = 0; c < P.nch;) {
                        const int sw = (P.nch - c >= 64 && P.sw_max >= 64) ? 64 : (P.nch - c >= 32 ? 32 : 16);
                        if (sw == 64) store_cols<64>(tacc + (uint32_t)c, stg, lane, ybase + c, P.ycols, rows_left);
                        else if (sw == 32) store_cols<32>(tacc + (uint32_t)c, stg, lane, ybase + c, P.ycols, rows_left);
                        else store_cols<16>(tacc + (uint32_t)c, stg, lane, ybase + c, P.ycols, rows_left);
                        c += sw;
                    }
                    if (sub == 0 && lane == 0) PROJ_TL(5, it);   // stored; about to release the slot
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarAccFree + slot));
                }
                if (++turn == ngroups) turn = 0;
                if (++slot == nslots) { slot = 0; slot_phase ^= 1; }
                col0 += P.nch;
                if (col0 == P.ycols) { col0 = 0; ++ti; }
            }
        }
    }
    if (!ok && lane == 0) atomicExch(P.status, 1);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

size_t smem_bytes(int K, int nch, int nchunks, int stages, int sw_max) {
    const size_t img = ((size_t)nchunks * (K / 8) * nch * 16 + 127) & ~(size_t)127;
    return img + (size_t)stages * K * 256 + 16 + 16 + kNumBars * 8 + 16 + (size_t)kEpiWarps * 32 * (sw_max * 2 + 16) + 128;
}

// Columns per chunk (one MMA shape: a multiple of 16, at most 256, dividing the columns of one tensor), chunks per
// launch, X stages (at least two) and the widest epilogue pass, such that everything fits shared memory.  Fewest
// launches win (every launch reads X again).
struct Plan { int nch, per_launch, stages, sw_max; };

bool make_plan(int c_in, int c_out, int nmat, Plan* plan) {
    bool found = false;
    long best_score = 0;
    for (int div = 1; div <= 16; ++div) {
        if (c_out % div != 0) continue;
        const int nch = c_out / div;
        if (nch > 256 || nch % 16 != 0) continue;
        const int total = (c_out / nch) * nmat;
        for (int sw = 64; sw >= 32; sw -= 32) {
            for (int stages = kMaxStages; stages >= 2; --stages) {
                int per = total;
                while (per >= 1 && smem_bytes(c_in, nch, per, stages, sw) > kMaxSmem) --per;
                if (per < 1) continue;
                const int launches = (total + per - 1) / per;
                // fewest launches; then up to four stages; then the wide pass; then more stages; then the wide chunk
                const long score = -(long)launches * 1000000 + (stages < 4 ? stages : 4) * 10000 + sw * 100 + stages * 10 + (nch > 128 ? 2 : nch > 64 ? 1 : 0);
                if (!found || score > best_score) {
                    found = true; best_score = score;
                    plan->nch = nch; plan->per_launch = per; plan->stages = stages; plan->sw_max = sw;
                }
            }
        }
    }
    return found;
}

}  // namespace

bool proj_supports(int c_in, int c_out) {
    Plan pl;
    return c_in >= 16 && c_in <= 256 && c_in % 16 == 0 && c_out >= 16 && c_out <= 256 && c_out % 16 == 0 &&
           make_plan(c_in, c_out, 1, &pl);
}

cudaError_t proj_setup() {
    if (!tensor_map_available()) return cudaErrorNotSupported;
    return cudaFuncSetAttribute(proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

cudaError_t launch_proj(const void* x, long long rows, int c_in, const float* w, int c_out, int nmat,
                        void* const* y, int* d_status, int num_sms, cudaStream_t stream)
{
    Plan pl;
    if (!proj_supports(c_in, c_out) || nmat < 1 || nmat > 3 || rows < 1 || rows > 0x7fffff00LL ||
        !make_plan(c_in, c_out, nmat, &pl))
        return cudaErrorInvalidValue;
    CUtensorMap map_x;
    if (!make_tile_map(&map_x, x, 2, 1, 1, (int)rows, c_in, 8, 128, 1)) return cudaErrorInvalidValue;

    const int total_chunks = (c_out / pl.nch) * nmat;
    const int ntiles = (int)((rows + 127) / 128);
    for (int c0 = 0; c0 < total_chunks; c0 += pl.per_launch) {
        const int nchunks = total_chunks - c0 < pl.per_launch ? total_chunks - c0 : pl.per_launch;
        ProjParams P;
        P.w = w;
        for (int i = 0; i < 3; ++i) P.y[i] = static_cast<__nv_bfloat16*>(i < nmat ? y[i] : nullptr);
        P.ycols = c_out; P.n0 = c0 * pl.nch;
        P.rows = (int)rows; P.K = c_in; P.nch = pl.nch; P.nchunks = nchunks; P.stages = pl.stages; P.sw_max = pl.sw_max;
        P.status = d_status;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(ntiles < num_sms ? ntiles : num_sms));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem_bytes(c_in, pl.nch, nchunks, pl.stages, pl.sw_max);
        cfg.stream = stream;
        // the launch may begin (barriers, tensor memory) while the kernel ahead of it in the stream drains; every
        // thread that reads global memory waits for that kernel first
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, proj_kernel, map_x, P);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace slide_attn

#ifdef SLIDE_ATTN_TIMELINE
// host [6][256]: per work item of CTA 0 the clock64 stamps listed at PROJ_TL; returns the cudaError_t of the copy
extern "C" int slide_attn_proj_timeline(long long* host) {
    return (int)cudaMemcpyFromSymbol(host, slide_attn::g_proj_timeline, sizeof(long long) * 6 * 256);
}
#endif
