// Shared device-side pieces of the GVA decode library: launch parameters, the split-KV work
// partition, the workspace layout, and small PTX wrappers.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gva.h"

namespace gva {

constexpr int kHeadsPerGroup = 4;   // H / G of every instantiated kernel
// Workspace header (ints): the partition of the flat tile list into units (for inspection) followed by one
// (first record, record count) pair per sequence, published by block 0 of the decode kernel for the combine kernel.
constexpr int kHdrInts = 8;
constexpr int kHdrTotal = 0;        // total tiles
constexpr int kHdrRanges = 1;       // equal contiguous ranges the tile list is cut into
constexpr int kHdrU = 2;            // tail units per range
constexpr int kHdrK = 3;            // tiles per tail unit
constexpr int kHdrEpoch = 4;        // stamp of the call whose header this is (handle serial and call number), written last
                                    // (release): a merge block that finds its own call's stamp here may use the header
                                    // before the decode grid is done.  What stands here before is the stamp of the last
                                    // call that used this workspace: another number of the same handle or another handle.
// Device-side scheduling state of one handle ("sync region": int32 words inside the library image).  Every call has an
// epoch number (1, 2, 3, ...); the call with epoch e uses the words of parity e & 1, and block 0 of its decode kernel
// clears the words of the other parity for the call after it, so nothing has to be reset at the end of a call and a
// call that gave up half-way leaves nothing behind that later calls would trip over.
constexpr int kSyncTicket = 0;      // [2] next tail unit to hand out
constexpr int kSyncWords = 2;       // (the fused decode step adds its own words behind these: see gva_decode_mma.cuh)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Everything a decode launch needs, passed by value.
struct DecodeParams {
    const void *v_pool;          // GVA: values.  GQA: values.
    const void *kr_pool;         // GVA: shared rotated positional keys.  GQA: unused.
    const void *k_pool;          // GQA only: keys.
    const int32_t *block_table;  // nullable
    const int32_t *seq_lens;
    const float *q;              // [B][H][d_q]
    int32_t *hdr;                // workspace header (kHdrInts + 2 B ints)
    float *rec_o;                // [n_rec][H * q_len][d_v] unnormalised partial outputs
    float *rec_ml;               // [n_rec][H * q_len][2]   running max (log2 domain) and sum
    float *out;                  // [B][H][d_v]
    float *lse;                  // nullable
    int32_t *dev_status;         // nullable
    int32_t *sync;               // this handle's sync region (see kSync*)
    int epoch;                   // this call's number on its handle (>= 1)
    int hdr_stamp;               // (handle serial % 2048) << 20 | call number % 2^20, + 1: see kHdrEpoch.  0 = none: a call that
                                 // is captured into a CUDA graph is replayed with the same number every time, so a header
                                 // left by the previous replay could not be told from this one's; nothing is fetched early then
    int n_rec;                   // records the workspace holds
    int B, H, G, P, num_pages, max_pages;
    int num_splits;              // 0 = balanced flat partition
    int rec_mult;                // partial records per (block, sequence): consumer warps per value group
    int early_start;             // 1: launched right behind step_front_kernel (see gva_decode_mma.cuh)
    const int32_t *append_pos;   // early_start: position being appended per sequence (its tile must not be read early)
    float scale_log2;            // softmax scale * log2(e)
    int q_len;                   // multi-token decode: new tokens per sequence (2..8; with cu_q: the most any sequence has); 0 or 1 otherwise
    const int32_t *cu_q;         // multi-token decode with a different count per sequence: first query row of every sequence ([B + 1]); else NULL
};

__device__ __forceinline__ void report_error(int32_t *dev_status, int code, int b) {
    if (dev_status) atomicCAS(dev_status, 0, code | (b << 8));
}

// ---- work partition --------------------------------------------------------------------------
// The cache stream of a batch is the concatenation of every sequence's tiles (TILE tokens each).
// s_off[b] = number of tiles before sequence b; s_off[B] = total.
//   balanced mode (num_splits == 0): the n_eff = ceil(total / ceil(total / gridDim.x)) leading thread
//     blocks take equal contiguous ranges of the flat tile list; block c, sequence b -> record c + b
//     (unique because c and b never decrease along the list and one of them grows at each cut).
//   uniform mode (num_splits == S): block c handles split c % S of sequence c / S -> record c.
// Must be called by every thread of the block; ends with a barrier.
template <int TILE>
__device__ __forceinline__ void compute_tile_offsets(const DecodeParams &p, int *s_off) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const long long cap = (long long)p.max_pages * p.P;
    for (int b = tid; b < p.B; b += nt) {
        int len = p.seq_lens[b];
        if (len < 0 || (long long)len > cap) {
            report_error(p.dev_status, GVA_ERR_SEQ_LEN, b);
            len = 0;
        }
        s_off[b + 1] = (len + TILE - 1) / TILE;
    }
    if (tid == 0) s_off[0] = 0;
    __syncthreads();
    if (tid < 32) {
        const int per = (p.B + 31) / 32;
        const int start = 1 + tid * per;
        const int end = min(start + per, p.B + 1);
        int sum = 0;
        for (int i = start; i < end; ++i) sum += s_off[i];
        int x = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, x, o);
            if (tid >= o) x += y;
        }
        int base = x - sum;
        for (int i = start; i < end; ++i) {
            base += s_off[i];
            s_off[i] = base;
        }
    }
    __syncthreads();
}

__host__ __device__ __forceinline__ int partitions_in_use(int total_tiles, int n_blocks) {
    if (total_tiles <= 0) return 0;
    int per = (total_tiles + n_blocks - 1) / n_blocks;
    return (total_tiles + per - 1) / per;
}
__host__ __device__ __forceinline__ int range_begin(int c, int total_tiles, int n_eff) {
    return (int)(((long long)c * total_tiles) / n_eff);
}
// block that owns flat tile x under range_begin(): the smallest c with range_begin(c+1) > x
__host__ __device__ __forceinline__ int range_owner(int x, int total_tiles, int n_eff) {
    return (int)((((long long)x + 1) * n_eff + total_tiles - 1) / total_tiles) - 1;
}

// ---- units ---------------------------------------------------------------------------------------
// Balanced mode cuts the flat tile list into n_ranges equal contiguous ranges (one per thread block), and
// each range into 1 + U units: a static head that its block always processes, and U tail units of K tiles
// each that are handed out through an atomic ticket to whichever block gets there first.  Blocks that stream
// slower than the rest therefore lose their tails to faster ones instead of setting the kernel time.
//   unit id  u = range * (U + 1) + j   (j = 0 head, j >= 1 tails): ordered by tile position, so the units that
//   intersect a sequence are one contiguous run, and (unit u, sequence b) -> record u + b is collision-free
//   (u and b never decrease along the tile list and one of them grows at every cut).
struct UnitPlan {
    int total, n_ranges, U, K;
};

// size of tail j (1-based): K, K/2, K/4, ... (at least 1), so the last pieces handed out are the smallest
__host__ __device__ __forceinline__ int tail_size(const UnitPlan &u, int j) {
    const int k = u.K >> (j - 1);
    return k > 0 ? k : 1;
}
__host__ __device__ __forceinline__ int tail_total(const UnitPlan &u) {
    int d = 0;
    for (int j = 1; j <= u.U; ++j) d += tail_size(u, j);
    return d;
}

__host__ __device__ __forceinline__ UnitPlan make_unit_plan(int total, int n_blocks, bool allow_dynamic) {
    UnitPlan u;
    u.total = total;
    u.n_ranges = partitions_in_use(total, n_blocks);
    u.U = 0;
    u.K = 1;
    const int per_block = total / (n_blocks > 0 ? n_blocks : 1);
#ifndef GVA_TAIL_DEN
#define GVA_TAIL_DEN 8      // build-time knobs: the first tail is 1/GVA_TAIL_DEN of a range, each next one half of that
                            // (measured on the long-context workload, gva_decode / step in us: 16 -> 91.2 / 93.5, 8 -> 90.85 / 92.9,
                            //  6 -> 91.2 / 93.1, 4 -> 91.5 / 93.3; two tails instead of three: the same; a fourth, single-tile tail: +0.7 / +0.4)
#define GVA_TAIL_UNITS 3
#endif
    if (allow_dynamic && per_block >= 8) {
        u.U = GVA_TAIL_UNITS;
        u.K = per_block / GVA_TAIL_DEN;
        if (u.K < 1) u.K = 1;
    }
    return u;
}
__host__ __device__ __forceinline__ int plan_units(const UnitPlan &u) { return u.n_ranges * (u.U + 1); }
// tiles [lo, hi) of unit (range c, part j)
__host__ __device__ __forceinline__ void unit_range(const UnitPlan &u, int c, int j, int &lo, int &hi) {
    const int r0 = range_begin(c, u.total, u.n_ranges), r1 = range_begin(c + 1, u.total, u.n_ranges);
    const int len = r1 - r0;
    const int dt = tail_total(u);
    const int d = len < dt ? len : dt;
    const int head = len - d;
    if (j == 0) {
        lo = r0;
        hi = r0 + head;
    } else {
        lo = r0 + head;
        for (int k = 1; k < j; ++k) lo += tail_size(u, k);
        hi = lo + tail_size(u, j);
        if (lo > r1) lo = r1;
        if (hi > r1) hi = r1;
    }
}
__host__ __device__ __forceinline__ int unit_of_tile(const UnitPlan &u, int x) {
    const int c = range_owner(x, u.total, u.n_ranges);
    const int r0 = range_begin(c, u.total, u.n_ranges), r1 = range_begin(c + 1, u.total, u.n_ranges);
    const int len = r1 - r0;
    const int dt = tail_total(u);
    const int d = len < dt ? len : dt;
    int rel = x - r0 - (len - d);
    if (rel < 0) return c * (u.U + 1);
    int j = 1;
    while (j < u.U && rel >= tail_size(u, j)) {
        rel -= tail_size(u, j);
        ++j;
    }
    return c * (u.U + 1) + j;
}
// upper bound on units for any total (for sizing the workspace)
__host__ __device__ __forceinline__ int unit_bound(int n_blocks) { return 5 * n_blocks; }

// This block's flat tile range and, in uniform mode, its fixed record.
struct BlockRange {
    int lo, hi;      // flat tiles [lo, hi)
    int rec_fixed;   // uniform mode: record index; balanced: -1
    int b_first;     // sequence containing tile lo (valid when lo < hi)
};

__device__ __forceinline__ int seq_of_tile(const int *s_off, int B, int x) {
    int lo = 0, hi = B - 1;   // largest b with s_off[b] <= x  (and s_off[b+1] > x because x < total)
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (s_off[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Static-only partition (CUDA-core kernel, and uniform mode of both kernels).
__device__ __forceinline__ BlockRange block_range(const DecodeParams &p, const int *s_off) {
    BlockRange r;
    const int total = s_off[p.B];
    if (p.num_splits > 0) {
        const int b = blockIdx.x / p.num_splits, s = blockIdx.x % p.num_splits;
        const int tiles = s_off[b + 1] - s_off[b];
        r.lo = s_off[b] + (int)(((long long)s * tiles) / p.num_splits);
        r.hi = s_off[b] + (int)(((long long)(s + 1) * tiles) / p.num_splits);
        r.rec_fixed = blockIdx.x;
        r.b_first = b;
    } else {
        const int n_eff = partitions_in_use(total, gridDim.x);
        r.rec_fixed = -1;
        if ((int)blockIdx.x >= n_eff) {
            r.lo = r.hi = 0;
            r.b_first = 0;
        } else {
            r.lo = range_begin(blockIdx.x, total, n_eff);
            r.hi = range_begin(blockIdx.x + 1, total, n_eff);
            r.b_first = (r.lo < r.hi) ? seq_of_tile(s_off, p.B, r.lo) : 0;
        }
    }
    return r;
}

// Block 0 of a decode kernel, threads [0, nt), after the block's dependency wait: clears the other parity's ticket and
// publishes the tile offsets and the unit plan for the combine kernel: per sequence the first record (per-warp
// multiplier applied) and the number of records of its run of units.
__device__ __forceinline__ void block0_duties(const DecodeParams &p, const int *s_off, const UnitPlan &plan, int tid, int nt) {
    if (blockIdx.x != 0 || tid >= nt) return;
    if (tid == 0) {
        p.sync[kSyncTicket + ((p.epoch & 1) ^ 1)] = 0;
        p.hdr[kHdrTotal] = plan.total;
        p.hdr[kHdrRanges] = plan.n_ranges;
        p.hdr[kHdrU] = plan.U;
        p.hdr[kHdrK] = plan.K;
    }
    for (int b = tid; b < p.B; b += nt) {
        int2 seg = make_int2(0, 0);
        if (p.num_splits > 0) {
            seg = make_int2(b * p.num_splits * p.rec_mult, p.num_splits * p.rec_mult);
        } else if (s_off[b + 1] > s_off[b]) {
            const int u0 = unit_of_tile(plan, s_off[b]), u1 = unit_of_tile(plan, s_off[b + 1] - 1);
            seg = make_int2((u0 + b) * p.rec_mult, (u1 - u0 + 1) * p.rec_mult);
        }
        reinterpret_cast<int2 *>(p.hdr + kHdrInts)[b] = seg;
    }
    // every one of the nt threads has stored its part (nt is a multiple of the warp size): publish the call's stamp
    asm volatile("bar.sync 1, %0;\n" ::"r"(nt) : "memory");
    if (tid == 0) asm volatile("st.release.gpu.global.b32 [%0], %1;\n" ::"l"(p.hdr + kHdrEpoch), "r"(p.hdr_stamp) : "memory");
}

// ---- optional in-kernel timeline (build with -DGVA_TRACE) ---------------------------------------------------
// Slots of %globaltimer stamps (ns), kept as a minimum (even slots) or a maximum (odd slots) over all threads that
// report; read and cleared by gva_debug_trace().  Compiled out of normal builds.
enum TraceSlot {
    kTrFrontEnterMin = 0, kTrFrontExitMax = 1, kTrDecodeEnterMin = 2, kTrDecodeEnterMax = 3, kTrFirstTileMin = 4,
    kTrFirstTileMax = 5, kTrLastTileMin = 6, kTrLastTileMax = 7, kTrArriveMin = 8, kTrArriveMax = 9, kTrCombineEnterMin = 10,
    kTrCombinePollMax = 11, kTrCombineOutMin = 12, kTrCombineOutMax = 13, kTrDecodeExitMin = 14, kTrDecodeExitMax = 15, kTrSlots = 16
};
constexpr int kTrCalls = 8;      // stamps of the last kTrCalls calls are kept apart (slot set = call number % kTrCalls)
#ifdef GVA_TRACE
__device__ unsigned long long g_trace[kTrCalls * kTrSlots];
__device__ __forceinline__ void trace(int slot, int call) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    unsigned long long *dst = &g_trace[(call % kTrCalls) * kTrSlots + slot];
    if (slot & 1) atomicMax(dst, t);
    else atomicMin(dst, t);
}
#else
__device__ __forceinline__ void trace(int, int) {}
#endif

// ---- small PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *ptr) {
    return (uint32_t)__cvta_generic_to_shared(ptr);
}
// 16-byte asynchronous global->shared copy; src_bytes == 0 writes 16 zero bytes instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// Programmatic dependent launch.  Every kernel of the library is launched with the
// "programmatic stream serialization" attribute and
//   - calls grid_dependency_launch() first, so the next kernel in the stream may be scheduled and run
//     its own set-up while this one works, and
//   - calls grid_dependency_wait() before its first global-memory access, which blocks until every
//     earlier kernel in the stream has completed and its writes are visible.
// Because each kernel waits before it touches memory (and so cannot finish before its predecessor),
// stream order is preserved for data; only launch latency and set-up overlap.  Kernels of other
// libraries never trigger early, so they are fully serialised as usual.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Host: launch with the programmatic-stream-serialization attribute (see above).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*fn)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, static_cast<KArgs>(args)...);
}

}  // namespace gva
