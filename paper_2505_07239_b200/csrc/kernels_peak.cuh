// Measured peaks of the two multiply pipes the gathered ring matmul can run on, for the roofline the benchmark
// reports against: a loop of the tensor-core instruction the limb kernel issues (tcgen05.mma kind::i8, M 128 x
// N 256 x K 32, u8 x u8 -> s32, operands resident in shared memory, accumulators in TMEM), and a loop of 64-bit
// multiply-adds on the integer ALUs (what the CUDA-core kernel's inner loop consists of).  Nothing here is part
// of the path: no global memory is read, and what is written is one word per thread so that the work stays live.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "kernels_limb.cuh"

namespace comet {
namespace peak {
constexpr int M = 128, N = 256, KC = 32;
constexpr int A_BYTES = M * KC, B_BYTES = N * KC;      // one operand tile each, K-major core-matrix layout
constexpr int BATCH = 32;                              // instructions per commit
constexpr int THREADS = 128;
constexpr int ALU_CHAINS = 8, ALU_THREADS = 1024;
}  // namespace peak

// One CTA per SM.  Thread 0 issues `batches` batches of 32 instructions, alternating between two accumulators of
// 256 columns and between two tiles per operand; a batch is committed to one of two mbarriers and the batch after
// the next one waits for it, so the pipe always has a full batch queued.  Every wait is bounded.
__global__ void __launch_bounds__(peak::THREADS, 1)
tensor_i8_probe_kernel(int batches, unsigned seed, int* error_flag, unsigned* sink) {
    using namespace peak;
    __shared__ __align__(128) uint8_t sA[2][A_BYTES];
    __shared__ __align__(128) uint8_t sB[2][B_BYTES];
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5;

    // operand bytes: a cheap hash, so that the multipliers see changing bits as they do on ring words
    for (int i = tid; i < (2 * A_BYTES + 2 * B_BYTES) / 4; i += THREADS) {
        unsigned v = (unsigned)i * 2654435761u + seed + blockIdx.x * 40503u;
        v ^= v >> 15; v *= 2246822519u; v ^= v >> 13;
        uint32_t* dst = i < 2 * A_BYTES / 4 ? reinterpret_cast<uint32_t*>(&sA[0][0]) + i
                                            : reinterpret_cast<uint32_t*>(&sB[0][0]) + (i - 2 * A_BYTES / 4);
        *dst = v;
    }
    ptx::fence_proxy_async_smem();           // the tensor core reads these bytes through the async proxy
    if (tid == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar[0]), 1);
        ptx::mbar_init(ptx::smem_u32(&bar[1]), 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_before_sync();
    __syncthreads();
    ptx::fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    if (tid == 0) {
        constexpr uint32_t IDESC = (2u << 4) | ((uint32_t)(M >> 4) << 24) | ((uint32_t)(N >> 3) << 17);
        const uint32_t a_lo[2] = {limb_desc_lo(ptx::smem_u32(&sA[0][0])), limb_desc_lo(ptx::smem_u32(&sA[1][0]))};
        const uint32_t b_lo[2] = {limb_desc_lo(ptx::smem_u32(&sB[0][0])), limb_desc_lo(ptx::smem_u32(&sB[1][0]))};
        const uint32_t bar0 = ptx::smem_u32(&bar[0]);
        bool ok = true;
        for (int b = 0; b < batches && ok; ++b) {
            if (b >= 2) ok = limb_wait(bar0 + 8 * (b & 1), (uint32_t)(((b - 2) >> 1) & 1), &abort_flag);
            if (!ok) break;
#pragma unroll
            for (int i = 0; i < BATCH; ++i)
                ptx::mma_i8(tmem_base + (i & 1) * N, a_lo[i & 1], LIMB_DESC_HI, b_lo[(i >> 1) & 1], LIMB_DESC_HI, IDESC,
                            (b == 0 && i < 2) ? 0u : 1u);
            ptx::mma_commit(bar0 + 8 * (b & 1));
        }
        // the last two batches
        for (int b = batches > 2 ? batches - 2 : 0; b < batches && ok; ++b)
            ok = limb_wait(bar0 + 8 * (b & 1), (uint32_t)((b >> 1) & 1), &abort_flag);
    }
    __syncthreads();
    if (warp == 0) {
        ptx::fence_after_sync();
        uint32_t d[8];
        ptx::tmem_ld8(tmem_base, d);
        ptx::tmem_wait_ld();
        if (sink && !abort_flag) sink[blockIdx.x * 32 + tid] = d[0] ^ d[7];
    }
    ptx::fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_flag) *error_flag = 1;
    if (warp == 0) {
        ptx::fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

// `iters` rounds of eight independent chains acc <- acc * a + b mod 2^64 per thread.
__global__ void __launch_bounds__(peak::ALU_THREADS)
alu_u64_probe_kernel(int iters, u64 seed, u64* sink) {
    using namespace peak;
    const u64 g = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    const u64 a = (seed * (2 * g + 1)) | 1ull, b = seed ^ (g * 0x9E3779B97F4A7C15ull);
    u64 acc[ALU_CHAINS];
#pragma unroll
    for (int j = 0; j < ALU_CHAINS; ++j) acc[j] = b + (u64)j * a;
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int j = 0; j < ALU_CHAINS; ++j) acc[j] = acc[j] * a + b;
    }
    u64 s = 0;
#pragma unroll
    for (int j = 0; j < ALU_CHAINS; ++j) s ^= acc[j];
    sink[g] = s;
}

}  // namespace comet
