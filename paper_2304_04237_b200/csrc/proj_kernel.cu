// Projections of a Slide-Attention block (Eq. 1: q = x W_q, k = x W_k, v = x W_v; Eq. 3: Concat(heads) W_o)
// as one persistent tcgen05 GEMM:  Y[rows x N] = X[rows x K] W[K x N], X and Y bf16 (token-major, channels
// contiguous), W given in fp32 and rounded to bf16 once by a prep launch, fp32 accumulation in tensor memory.
//
// The column range of one launch is split into chunks of `nch` columns (one MMA shape); all chunk images of the
// launch stay resident in shared memory, X comes in as 128-row tiles through a TMA ring.  K <= 256 is one tile
// deep, so a work item (row tile, chunk) is K/16 MMAs of M = 128, N = nch, followed by one commit.
//
// Shared-memory operand layout (no swizzle, K-major core matrices of 8 rows x 16 bytes):
//   X tile   [K/8][128 rows][16 B]   written by K/8 TMA boxes of 8 channels x 128 rows (rows past the end read 0)
//   W chunk  [K/8][nch cols][16 B]   written by the prep kernel, copied in with one bulk copy per launch
//
// Warps: 0 TMA producer, 1 MMA issuer (owns tensor memory), 2-5 epilogue (TMEM lane quarter = warp % 4: one
// thread per output row, tcgen05.ld.32x32b -> bf16 -> 16-byte stores).  Two accumulator slots of 256 columns let
// the MMAs of item i+1 run under the epilogue of item i.  Every wait is bounded; a wait that runs out sets the
// status word and the kernel still releases tensor memory.
#include "common.cuh"
#include "ptx.cuh"

namespace slide_attn {

namespace {

constexpr int kThreads = 192;
constexpr int kMaxStages = 6;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSlotCols = 256;
constexpr size_t kMaxSmem = 227 * 1024;
constexpr size_t kMaxImage = 96 * 1024;      // resident weight chunks of one launch

constexpr int kBarXFull = 0;                 // [kMaxStages]
constexpr int kBarXEmpty = kMaxStages;       // [kMaxStages]  one arrival: the commit behind the tile's last MMA
constexpr int kBarWeights = 2 * kMaxStages;
constexpr int kBarAccFull = kBarWeights + 1; // [2]
constexpr int kBarAccFree = kBarAccFull + 2; // [2]  count 4 (epilogue warps)
constexpr int kNumBars = kBarAccFree + 2;

struct ProjParams {
    const unsigned char* img;    // chunk images of this launch, chunk after chunk
    __nv_bfloat16* y[3];         // output tensors, each [rows][ycols]
    int ycols;                   // channels of one output tensor
    int n0;                      // first column of this launch, counted over the concatenated output tensors
    int rows, K, nch, nchunks, stages;
    int* status;
};

__device__ __forceinline__ void tmem_ld_32x32b_x16_wait(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}

// bf16 images of the weights, one per chunk of nch columns: [chunk][K/8][nch][8 K-consecutive bf16].
// `w` holds `nmat` row-major [K][ncols] fp32 matrices one after the other; output column n of the concatenation
// is column n % ncols of matrix n / ncols.
__global__ void __launch_bounds__(256)
proj_prep_kernel(const float* __restrict__ w, int K, int ncols, int nmat, int nch, unsigned char* __restrict__ img)
{
    grid_launch_dependents();
    const int ntot = ncols * nmat, kgs = K >> 3;
    const size_t chunk_bytes = (size_t)kgs * nch * 16;
    for (int item = blockIdx.x * blockDim.x + threadIdx.x; item < kgs * ntot; item += gridDim.x * blockDim.x) {
        const int kg = item / ntot, n = item - kg * ntot;
        const float* src = w + (size_t)(n / ncols) * K * ncols + (size_t)(8 * kg) * ncols + (n % ncols);
        float val[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) val[e] = src[(size_t)e * ncols];
        unsigned char* dst = img + (size_t)(n / nch) * chunk_bytes + ((size_t)kg * nch + (n % nch)) * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16(val[0], val[1]), pack_bf16(val[2], val[3]),
                                                    pack_bf16(val[4], val[5]), pack_bf16(val[6], val[7]));
    }
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
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int ntiles = (P.rows + 127) >> 7;
    const int my_tiles = (int)blockIdx.x < ntiles ? (ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int S = P.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init_only(bar(kBarXFull + s), 1); mbar_init_only(bar(kBarXEmpty + s), 1); }
        mbar_init_only(bar(kBarWeights), 1);
        for (int i = 0; i < 2; ++i) { mbar_init_only(bar(kBarAccFull + i), 1); mbar_init_only(bar(kBarAccFree + i), 4); }
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(smem + tmem_off), kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<const volatile uint32_t*>(smem + tmem_off);
    bool ok = true;

    if (warp == 0) {
        // ---- TMA producer: the weight images once, then the X tiles of this CTA through the ring.  Everything
        // this kernel reads from global memory is read here, after the kernels ahead of it in the stream have
        // completed (the kernel may have been launched before they did).
        uint32_t leader;
        if (elect_one(leader) && my_tiles > 0) {
            grid_dependency_wait();
            mbar_expect_tx(bar(kBarWeights), img_bytes);
            bulk_load_1d(smem_u32(smem), P.img, img_bytes, bar(kBarWeights));
            for (int t = 0; ok && t < my_tiles; ++t) {
                const int s = t % S, m = (int)blockIdx.x + t * (int)gridDim.x;
                if (!mbar_wait(bar(kBarXEmpty + s), (uint32_t)(((t / S) & 1) ^ 1))) { ok = false; break; }
                const uint32_t dst = smem_u32(smem + x_off + (size_t)s * stage_bytes), fb = bar(kBarXFull + s);
                mbar_expect_tx(fb, stage_bytes);
                for (int kg = 0; kg < (P.K >> 3); ++kg) tma_load_4d(dst + (uint32_t)kg * 2048u, &map_x, fb, 8 * kg, m * 128, 0, 0);
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
            int it = 0;
            for (int t = 0; ok && t < my_tiles; ++t) {
                const int s = t % S;
                if (!mbar_wait(bar(kBarXFull + s), (uint32_t)((t / S) & 1))) { ok = false; break; }
                const uint32_t sX = smem_u32(smem + x_off + (size_t)s * stage_bytes);
                for (int ch = 0; ch < P.nchunks; ++ch, ++it) {
                    const int slot = it & 1;
                    if (!mbar_wait(bar(kBarAccFree + slot), (uint32_t)(((it >> 1) & 1) ^ 1))) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t dcol = tmem + (uint32_t)slot * kSlotCols;
                    const uint32_t sB = sB0 + (uint32_t)ch * chunk_bytes;
                    for (int kk = 0; kk < (P.K >> 4); ++kk)
                        umma_bf16_ss(dcol, umma_smem_desc(sX + (uint32_t)kk * 4096u, 2048, 128),
                                     umma_smem_desc(sB + (uint32_t)kk * 2u * b_lbo, b_lbo, 128), idesc, kk > 0 ? 1u : 0u);
                    umma_commit(bar(kBarAccFull + slot));
                }
                if (ok) umma_commit(bar(kBarXEmpty + s));       // the tile's last MMA has read it
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, leader) != 0;
    } else {
        // ---- epilogue: thread = output row 32 (warp % 4) + lane of the tile
        const int sub = warp & 3;
        const uint32_t tlane = tmem + ((uint32_t)(32 * sub) << 16);
        int it = 0;
        for (int t = 0; ok && t < my_tiles; ++t) {
            const long long row = ((long long)blockIdx.x + (long long)t * gridDim.x) * 128 + 32 * sub + lane;
            const bool live = row < (long long)P.rows;
            for (int ch = 0; ch < P.nchunks; ++ch, ++it) {
                const int slot = it & 1;
                if (!warp_wait(bar(kBarAccFull + slot), (uint32_t)((it >> 1) & 1))) { ok = false; break; }
                tc_fence_after_sync();
                for (int c = 0; c < P.nch; c += 16) {
                    float a[16];
                    tmem_ld_32x32b_x16_wait(tlane + (uint32_t)slot * kSlotCols + (uint32_t)c, a);
                    const int n = P.n0 + ch * P.nch + c;                 // 16 columns never straddle two tensors
                    const int ti = n / P.ycols, col = n - ti * P.ycols;
                    if (live) {
                        uint4* dst = reinterpret_cast<uint4*>(P.y[ti] + (size_t)row * P.ycols + col);
                        dst[0] = make_uint4(pack_bf16(a[0], a[1]), pack_bf16(a[2], a[3]), pack_bf16(a[4], a[5]), pack_bf16(a[6], a[7]));
                        dst[1] = make_uint4(pack_bf16(a[8], a[9]), pack_bf16(a[10], a[11]), pack_bf16(a[12], a[13]), pack_bf16(a[14], a[15]));
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAccFree + slot));
            }
        }
    }
    if (!ok && lane == 0) atomicExch(P.status, 1);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

size_t smem_bytes(int K, int nch, int nchunks, int stages) {
    const size_t img = ((size_t)nchunks * (K / 8) * nch * 16 + 127) & ~(size_t)127;
    return img + (size_t)stages * K * 256 + 16 + 16 + kNumBars * 8 + 128;
}

}  // namespace

bool proj_supports(int c_in, int c_out) {
    return c_in >= 16 && c_in <= 256 && c_in % 16 == 0 && c_out >= 16 && c_out <= 256 && c_out % 16 == 0;
}

// columns per chunk: the whole tensor when its image fits the resident budget, else half of it
static int chunk_cols(int c_in, int c_out) {
    if ((size_t)c_in * c_out * 2 <= kMaxImage) return c_out;
    return (c_out / 2) % 16 == 0 ? c_out / 2 : 0;
}

size_t proj_workspace_bytes(int c_in, int c_out, int nmat) { return (size_t)c_in * c_out * nmat * 2; }

cudaError_t proj_setup() {
    if (!tensor_map_available()) return cudaErrorNotSupported;
    return cudaFuncSetAttribute(proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
}

cudaError_t launch_proj(const void* x, long long rows, int c_in, const float* w, int c_out, int nmat,
                        void* const* y, void* workspace, int* d_status, int num_sms, cudaStream_t stream)
{
    if (!proj_supports(c_in, c_out) || nmat < 1 || nmat > 3 || rows < 1 || rows > 0x7fffff00LL) return cudaErrorInvalidValue;
    const int nch = chunk_cols(c_in, c_out);
    if (nch == 0) return cudaErrorInvalidValue;
    unsigned char* img = static_cast<unsigned char*>(workspace);
    const int ntot = c_out * nmat;
    {
        const int items = (c_in / 8) * ntot;
        proj_prep_kernel<<<(items + 255) / 256, 256, 0, stream>>>(w, c_in, c_out, nmat, nch, img);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    CUtensorMap map_x;
    if (!make_tile_map(&map_x, x, 2, 1, 1, (int)rows, c_in, 8, 128, 1)) return cudaErrorInvalidValue;

    const size_t chunk_bytes = (size_t)(c_in / 8) * nch * 16;
    const int total_chunks = ntot / nch;
    int per_launch = (int)(kMaxImage / chunk_bytes);
    if (per_launch < 1) return cudaErrorInvalidValue;
    if (per_launch > total_chunks) per_launch = total_chunks;
    const int ntiles = (int)((rows + 127) / 128);
    bool first = true;
    for (int c0 = 0; c0 < total_chunks; c0 += per_launch) {
        const int nchunks = total_chunks - c0 < per_launch ? total_chunks - c0 : per_launch;
        int stages = kMaxStages;
        while (stages >= 2 && smem_bytes(c_in, nch, nchunks, stages) > kMaxSmem) --stages;
        if (stages < 2) return cudaErrorInvalidConfiguration;
        ProjParams P;
        P.img = img + (size_t)c0 * chunk_bytes;
        for (int i = 0; i < 3; ++i) P.y[i] = static_cast<__nv_bfloat16*>(i < nmat ? y[i] : nullptr);
        P.ycols = c_out; P.n0 = c0 * nch;
        P.rows = (int)rows; P.K = c_in; P.nch = nch; P.nchunks = nchunks; P.stages = stages;
        P.status = d_status;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(ntiles < num_sms ? ntiles : num_sms));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem_bytes(c_in, nch, nchunks, stages);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = first ? 1 : 0;          // only the launch right behind the prep kernel overlaps it
        first = false;
        cudaError_t e = cudaLaunchKernelEx(&cfg, proj_kernel, map_x, P);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace slide_attn
