// Microbenchmark behind the prefill kernel's design: how fast does an SM take tcgen05.mma (M = 128, K = 16, bf16,
// f32 accumulate) for several N, with A in shared or tensor memory, from one or two issuing threads per block and
// one or two blocks per SM?  Operands are constant garbage; only the timing matters.  Build and run on a B200:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -DGVA_WITH_MMA umma_bench.cu -o umma_bench -lcuda && ./umma_bench
// Every wait is bounded, and tensor memory is freed on every path.
#include <cstdio>

#include "gva_prefill.cuh"
using namespace gva;

__global__ void __launch_bounds__(128) umma_rate_kernel(int N, int reps, int issuers, int a_in_tmem, long long *out) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bar[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort;
    const uint32_t sb = smem_u32(smem);
    for (int i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(smem)[i] = 0x3c003c00u;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar[0]), 1);
        mbar_init(smem_u32(&bar[1]), 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (threadIdx.x < 32) {
        tmem_alloc(smem_u32(&s_tmem), 256);
        tmem_relinquish();
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0 && w < issuers) {
        const uint32_t idesc = umma_idesc(128, N, false);
        const uint64_t a = smem_desc(sb, 16, 1024, kSwz128), b = smem_desc(sb + 16384 + w * 8192, 16, 1024, kSwz128);
        const uint32_t d = issuers == 2 ? tmem + w * 64 : tmem;      // one accumulator per issuer
        const long long t0 = clock64();
        for (int r = 0; r < reps; r += 8) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (a_in_tmem) umma_bf16_ts(d, tmem + 192, b + (u & 3) * 2, idesc, 1);
                else umma_bf16(d, a + (u & 3) * 2, b + (u & 3) * 2, idesc, 1);
            }
        }
        umma_commit(smem_u32(&bar[w]));
        const bool ok = mbar_wait_bounded(smem_u32(&bar[w]), 0, &s_abort);
        const long long t1 = clock64();
        if (blockIdx.x == 0 && w == 0) {
            out[0] = t1 - t0;
            out[1] = ok;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) {
        tc_fence_after();
        tmem_dealloc(tmem, 256);
    }
}

int main() {
    long long *d, h[2];
    if (cudaMalloc(&d, 64) != cudaSuccess) return 1;
    cudaFuncSetAttribute(umma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    const int reps = 4000;
    printf("blocks/SM  issuers/block  A        N    cycles per MMA per issuer   cycles per MMA per SM\n");
    for (int bps = 1; bps <= 2; ++bps)
        for (int a_in_tmem = 0; a_in_tmem < 2; ++a_in_tmem)
            for (int issuers = 1; issuers <= 2; ++issuers)
                for (int N : {64, 128, 256}) {
                    if (issuers == 2 && N > 64) continue;                 // two accumulators of N columns each must fit below column 192
                    const size_t smem = bps == 1 ? 100 * 1024 : 52 * 1024;   // the request decides how many blocks share an SM
                    umma_rate_kernel<<<148 * bps, 128, smem>>>(N, reps, issuers, a_in_tmem, d);
                    const cudaError_t e = cudaDeviceSynchronize();
                    cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
                    printf("%9d  %13d  %-7s  %3d  %26.1f  %22.1f  %s%s\n", bps, issuers, a_in_tmem ? "tmem" : "smem", N, (double)h[0] / reps,
                           (double)h[0] / reps / (issuers * bps), h[1] ? "" : "TIMEOUT ", e == cudaSuccess ? "" : cudaGetErrorString(e));
                }
    cudaFree(d);
    return 0;
}
