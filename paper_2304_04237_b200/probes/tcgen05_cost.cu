// Stand-alone probe of the costs the persistent kernel's schedule rests on (one CTA, valid
// instructions only, every wait bounded):
//   1. back-to-back tcgen05.mma (M = 128, K = 16, bf16 -> fp32), fully unrolled so that the issuing
//      thread executes nothing else: cycles per instruction as a function of N, of the A operand's
//      home (shared memory / tensor memory), of the number of accumulator tiles the sequence
//      alternates between, of the shared-memory layout of the operands and of the number of issuing threads; and the latency from the last issue
//      to the wake-up of a thread waiting on the commit barrier
//   2. tensor-memory loads and stores (issue -> wait complete) for one warp
//   3. a wait on an mbarrier phase that is already complete, in the forms the kernels could use, each
//      measured as a chain of 64 in which the next probe starts only after a branch on the last result
// Build: python -m paper_2304_04237_b200.build --probes      Run: paper_2304_04237_b200/probes/_build/tcgen05_cost
#include <cstdio>
#include <cstdlib>

#include "ptx.cuh"
using namespace slide_attn;

struct Res { long long issue, total; int ok; };

template <int MODE, int N, int NT, int COUNT, int ISSUERS>
__global__ void __launch_bounds__(192, 1) mma_seq(Res* res)
{
    __shared__ __align__(1024) unsigned char sA[4096];
    __shared__ __align__(1024) unsigned char sB[256 * 32];
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 4096 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(sA)[i] = 0x3c003c00u + (i & 7);
    for (int i = threadIdx.x; i < 256 * 32 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(sB)[i] = 0x3c003c00u + (i & 15);
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bars[0]), 1); mbar_init(smem_u32(&bars[1]), 1); }
    if (warp == 4) tmem_alloc(smem_u32(&tmem_slot), 512);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    if (warp < 4) {                                   // clear every column the run touches
        uint32_t z[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) z[i] = 0u;
        for (int c = 0; c < 512; c += 16) tmem_st_32x32b_x16(tmem + ((uint32_t)(32 * warp) << 16) + c, z);
        tmem_wait_st();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 4 || (ISSUERS == 2 && warp == 5)) {
        const int me = warp - 4;
        uint32_t leader;
        if (elect_one(leader)) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, N);
            // MODE 0: the two K-halves of an 8-row group lie side by side (LBO 128, SBO 256);
            // MODE 2: K-halves as separate planes of all rows (A: LBO 2048, SBO 128; B: LBO 16 N, SBO 128)
            const uint64_t adesc = MODE == 2 ? umma_smem_desc(smem_u32(sA), 2048, 128) : umma_smem_desc(smem_u32(sA), 128, 256);
            const uint64_t bdesc = MODE == 2 ? umma_smem_desc(smem_u32(sB), 16 * N, 128) : umma_smem_desc(smem_u32(sB), 128, 256);
            const uint32_t acol = tmem + 504;        // A operand of the .ts form: 8 columns
            const uint32_t bar = smem_u32(&bars[me]);
            const uint32_t d0 = tmem + (uint32_t)(me * NT * N);
            const long long t0 = clock64();
#pragma unroll
            for (int i = 0; i < COUNT; ++i) {
                if (MODE != 1) umma_bf16_ss(d0 + (uint32_t)((i % NT) * N), adesc, bdesc, idesc, i >= NT ? 1u : 0u);
                else umma_bf16_ts(d0 + (uint32_t)((i % NT) * N), acol, bdesc, idesc, i >= NT ? 1u : 0u);
            }
            const long long t1 = clock64();
            umma_commit(bar);
            const bool ok = mbar_wait(bar, 0);
            const long long t2 = clock64();
            res[me].issue = t1 - t0;
            res[me].total = t2 - t0;
            res[me].ok = ok ? 1 : 0;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

__global__ void __launch_bounds__(160, 1) tmem_latency(long long* out)
{
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 4) tmem_alloc(smem_u32(&tmem_slot), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    if (warp < 4) {
        const uint32_t tq = tmem + ((uint32_t)(32 * warp) << 16);
        uint32_t z[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) z[i] = lane + i;
        for (int c = 0; c < 512; c += 16) tmem_st_32x32b_x16(tq + c, z);
        tmem_wait_st();
        __syncwarp();
        for (int rep = 0; rep < 3; ++rep) {
            float v[32];
            const long long a = clock64();
            tmem_ld_32x32b_x32(tq, v);
            const long long b = clock64();
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) s += v[i];
            if (s == 12345.f) out[63] = 1;
            if (lane == 0 && warp == 0) out[0 * 4 + rep] = b - a;
        }
        for (int rep = 0; rep < 3; ++rep) {
            uint32_t r[48];
            const long long a = clock64();
            tmem_ld3_16x256b_x4_nowait(tq, tq + 32, tq + 64, r);
            tmem_wait_ld48(r);
            const long long b = clock64();
            uint32_t s = 0;
#pragma unroll
            for (int i = 0; i < 48; ++i) s += r[i];
            if (s == 12345u) out[63] = 1;
            if (lane == 0 && warp == 0) out[1 * 4 + rep] = b - a;
        }
        for (int rep = 0; rep < 3; ++rep) {
            const long long a = clock64();
            tmem_st_32x32b_x16(tq + 64, z);
            tmem_wait_st();
            const long long b = clock64();
            if (lane == 0 && warp == 0) out[2 * 4 + rep] = b - a;
        }
        for (int rep = 0; rep < 3; ++rep) {
            uint32_t r8[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) r8[i] = z[i];
            const long long a = clock64();
            tmem_st_16x256b_x2(tq + 96, r8);
            tmem_st_16x256b_x2(tq + 112, r8);
            tmem_st_16x256b_x2(tq + 128, r8);
            tmem_wait_st();
            const long long b = clock64();
            if (lane == 0 && warp == 0) out[3 * 4 + rep] = b - a;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

__device__ __forceinline__ bool try_wait_hint(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(100000u) : "memory");
    return done != 0;
}
__device__ __forceinline__ bool try_wait_nohint(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

__global__ void wait_cost(long long* out)
{
    __shared__ __align__(8) unsigned long long bars[8];
    const int lane = threadIdx.x & 31;
    const uint32_t b0 = smem_u32(&bars[0]);
    if (threadIdx.x == 0) for (int i = 0; i < 8; ++i) mbar_init(b0 + 8 * i, 1);
    __syncthreads();
    if (threadIdx.x == 0) for (int i = 0; i < 8; ++i) mbar_arrive(b0 + 8 * i);   // phase 0 of each is complete
    __syncthreads();
    int acc = 0;
    long long a, b;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { if (!try_wait_hint(b0 + 8 * (i & 7), 0)) break; ++acc; }
    b = clock64(); if (lane == 0) out[0] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { if (!__all_sync(0xffffffffu, try_wait_hint(b0 + 8 * (i & 7), 0) ? 1 : 0)) break; ++acc; }
    b = clock64(); if (lane == 0) out[1] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { if (!try_wait_nohint(b0 + 8 * (i & 7), 0)) break; ++acc; }
    b = clock64(); if (lane == 0) out[2] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { if (!mbar_test(b0 + 8 * (i & 7), 0)) break; ++acc; }
    b = clock64(); if (lane == 0) out[3] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { __syncwarp(); if (lane == 0) mbar_arrive(b0 + 40); }
    b = clock64(); if (lane == 0) out[4] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { if (!__all_sync(0xffffffffu, acc)) break; ++acc; }
    b = clock64(); if (lane == 0) out[5] = (b - a) / 64;
    a = clock64();
#pragma unroll 1
    for (int i = 0; i < 64; ++i) { ++acc; asm volatile("" : "+r"(acc)); }
    b = clock64(); if (lane == 0) out[6] = (b - a) / 64;
    if (acc == 12345) out[15] = acc;
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at line %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)

template <int MODE, int N, int NT, int COUNT, int ISSUERS>
void run(Res* d)
{
    static_assert(ISSUERS * NT * N <= 496, "tensor memory");
    Res h[2];
    for (int rep = 0; rep < 3; ++rep) {
        CK(cudaMemset(d, 0, 2 * sizeof(Res)));
        mma_seq<MODE, N, NT, COUNT, ISSUERS><<<1, 192>>>(d);
        CK(cudaDeviceSynchronize());
    }
    CK(cudaMemcpy(h, d, sizeof(h), cudaMemcpyDeviceToHost));
    for (int me = 0; me < ISSUERS; ++me)
        printf("| %s | %3d | %d | %3d | %d | %6lld | %6lld | %6.1f | %6lld | %d |\n", MODE == 1 ? "tensor memory" : MODE == 2 ? "shared memory, K-halves as planes" : "shared memory", N, NT, COUNT,
               ISSUERS, h[me].issue, h[me].total, (double)h[me].issue / COUNT, h[me].total - h[me].issue, h[me].ok);
}

int main()
{
    Res* d; CK(cudaMalloc(&d, 2 * sizeof(Res)));
    printf("| A operand | N | accumulator tiles | MMAs | issuing threads | issue cycles | cycles to wake-up | cycles per MMA | commit -> wake-up | ok |\n|---|---|---|---|---|---|---|---|---|---|\n");
    run<1, 16, 1, 72, 1>(d);  run<1, 32, 1, 18, 1>(d);  run<1, 32, 1, 72, 1>(d);  run<1, 32, 2, 72, 1>(d);  run<1, 32, 4, 72, 1>(d);
    run<1, 64, 1, 72, 1>(d);  run<1, 64, 2, 72, 1>(d);  run<1, 96, 1, 72, 1>(d);  run<1, 96, 2, 72, 1>(d);  run<1, 112, 1, 72, 1>(d);
    run<1, 128, 1, 72, 1>(d); run<1, 256, 1, 72, 1>(d);
    run<0, 32, 1, 72, 1>(d);  run<0, 32, 2, 72, 1>(d);  run<0, 64, 1, 72, 1>(d);  run<0, 96, 1, 72, 1>(d);
    run<0, 128, 1, 72, 1>(d); run<0, 192, 1, 72, 1>(d); run<0, 256, 1, 72, 1>(d);
    run<2, 32, 1, 72, 1>(d);  run<2, 64, 1, 72, 1>(d);  run<2, 128, 1, 72, 1>(d); run<2, 192, 1, 72, 1>(d); run<2, 256, 1, 72, 1>(d);
    run<1, 32, 1, 72, 2>(d);  run<1, 96, 1, 72, 2>(d);  run<0, 32, 1, 72, 2>(d);
    run<1, 32, 1, 3, 1>(d);   run<1, 96, 1, 2, 1>(d);

    long long* d_t; CK(cudaMalloc(&d_t, 64 * sizeof(long long))); CK(cudaMemset(d_t, 0, 64 * sizeof(long long)));
    tmem_latency<<<1, 160>>>(d_t);
    CK(cudaDeviceSynchronize());
    long long ht[64]; CK(cudaMemcpy(ht, d_t, sizeof(ht), cudaMemcpyDeviceToHost));
    const char* names[4] = {"tcgen05.ld.32x32b.x32 + wait", "3 x tcgen05.ld.16x256b.x4 + wait", "tcgen05.st.32x32b.x16 + wait", "3 x tcgen05.st.16x256b.x2 + wait"};
    printf("\n| tensor-memory access (one warp, cycles, three repeats) | | | |\n|---|---|---|---|\n");
    for (int k = 0; k < 4; ++k) printf("| %s | %lld | %lld | %lld |\n", names[k], ht[k * 4], ht[k * 4 + 1], ht[k * 4 + 2]);

    CK(cudaMemset(d_t, 0, 64 * sizeof(long long)));
    wait_cost<<<1, 32>>>(d_t);
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(ht, d_t, sizeof(ht), cudaMemcpyDeviceToHost));
    const char* wn[7] = {"mbarrier.try_wait with a time hint", "the same + warp vote", "mbarrier.try_wait without a hint", "mbarrier.test_wait",
                         "__syncwarp + lane-0 arrive", "warp vote alone", "empty loop (to subtract)"};
    printf("\n| completed-phase wait, per link of a dependent chain | cycles |\n|---|---|\n");
    for (int k = 0; k < 7; ++k) printf("| %s | %lld |\n", wn[k], ht[k]);
    return 0;
}
