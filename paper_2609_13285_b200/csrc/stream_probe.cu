// Read-only streaming probe: how fast can this GPU pull a buffer out of HBM once, when nothing is computed?
//
// Harness code for the benchmark, not part of the library's C ABI (it is built into its own small shared object):
// bench.py times it over a buffer of the same size as the cache it benchmarks, next to the decode kernel, so that the
// decode kernel's rate can be read against a read-only ceiling measured in the same run as well as against the copy
// bandwidth (which moves every byte twice).  The access pattern is the decode kernel's own: bulk asynchronous copies
// into a shared-memory ring, two resident blocks per SM, each block over one contiguous share of the buffer, with the
// same evict-first L2 policy; a second thread merely touches each landed chunk and hands the slot back.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kChunk = 32768;      // bytes per bulk copy (the decode kernel moves ~34 KB per tile)
constexpr int kStages = 3;
constexpr unsigned kSpinLimit = 1u << 26;      // polls before a wait gives up (tens of milliseconds)

__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool wait_parity(uint64_t *bar, uint32_t parity) {
    for (unsigned it = 0; it < kSpinLimit; ++it) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(ok)
                     : "r"(s32(bar)), "r"(parity)
                     : "memory");
        if (ok) return true;
    }
    return false;
}

__global__ void __launch_bounds__(64) stream_read_kernel(const unsigned char *__restrict__ src, size_t bytes, int *status) {
    extern __shared__ __align__(1024) unsigned char ring[];
    __shared__ __align__(8) uint64_t full[kStages], empty[kStages];
    __shared__ int s_abort;
    const size_t n_chunks = bytes / kChunk;
    const size_t per = (n_chunks + gridDim.x - 1) / gridDim.x;
    const size_t lo = per * blockIdx.x, hi = lo + per < n_chunks ? lo + per : n_chunks;
    const int n = hi > lo ? (int)(hi - lo) : 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(s32(&full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(s32(&empty[s])));
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t pol;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
        int issued = 0;
        for (int i = 0; i < n; ++i) {
            const int st = i % kStages;
            if (!wait_parity(&empty[st], ((i / kStages) & 1) ^ 1)) {
                s_abort = 1;
                atomicExch(status, 1);
                break;
            }
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(s32(&full[st])), "r"(kChunk) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::"r"(
                             s32(ring + (size_t)st * kChunk)),
                         "l"(src + (lo + i) * kChunk), "r"(kChunk), "r"(s32(&full[st])), "l"(pol)
                         : "memory");
            ++issued;
        }
        if (s_abort)      // copies in flight must land before the block's shared memory is released
            for (int i = issued > kStages ? issued - kStages : 0; i < issued; ++i) wait_parity(&full[i % kStages], (i / kStages) & 1);
    } else if (threadIdx.x == 32) {
        unsigned acc = 0;
        for (int i = 0; i < n; ++i) {
            const int st = i % kStages;
            if (!wait_parity(&full[st], (i / kStages) & 1) || *(volatile int *)&s_abort) {
                atomicExch(status, 1);
                break;
            }
            acc ^= *reinterpret_cast<volatile unsigned *>(ring + (size_t)st * kChunk);
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(s32(&empty[st])) : "memory");
        }
        if (acc == 0x12345678u) atomicExch(status, 2);      // keeps the read alive; never true for the benchmark's buffers in practice
    }
    __syncthreads();
}

}  // namespace

// Enqueues one read of `bytes` bytes (rounded down to a multiple of 32 KB) starting at the 16-byte aligned device
// pointer `src` on `stream`; *status (device int32, caller-zeroed) becomes non-zero if a bounded wait expired.
// Returns 0, or 1 if the launch failed.
extern "C" int gva_probe_stream_read(const void *src, size_t bytes, int *status, void *stream) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(stream_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStages * kChunk) != cudaSuccess) return 1;
        attr_set = true;
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 1;
    stream_read_kernel<<<2 * sms, 64, kStages * kChunk, static_cast<cudaStream_t>(stream)>>>(static_cast<const unsigned char *>(src), bytes, status);
    return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
