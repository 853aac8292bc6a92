// Tensor-core split-KV decode kernel over the paged bf16 GVA cache (sm_100a).
//
// Why tensor cores at all: per cached token the path needs 4 heads x (d_v + d_r + d_v) multiply-adds
// per group on 2-byte elements, about 8.5 flop per byte.  On CUDA cores that is more issue slots than
// an SM has at the HBM rate; on the tensor pipe it is a few percent.
//
// Layout of the work
//   thread block = contiguous range of TILE-token tiles of the batch's cache stream (see gva_common.cuh)
//   warp g < G   = consumer of value group g (its 4 query heads);  warp G = producer (one elected lane)
//   producer     : TMA (cp.async.bulk.tensor.2d) loads of the G value tiles and the shared positional-key
//                  tile of each cache tile into an NSTAGE ring, completion on mbarriers; 128-byte
//                  swizzle so that ldmatrix is bank-conflict free
//   consumer     : S^T[token, col] = V_tile . Q^T  with mma.sync.m16n8k16 (bf16 in, f32 accumulate):
//                  M = 16 tokens, K = value dims then RoPE dims, N = 8 columns = 4 heads x {hi, lo};
//                  the absorbed f32 query is split q = hi + lo into two bf16 numbers, so the otherwise
//                  idle half of the N dimension carries the low-order bits and the score keeps ~16
//                  mantissa bits of q.  Online softmax (base 2) down the token rows with warp shuffles.
//                  P is split the same way, transposed in registers with movmatrix, and
//                  O^T[dim, col] += V_tile^T . P^T uses the same shared-memory tile through
//                  ldmatrix.trans.  Each value byte is read from HBM once and serves all 4 heads.
//   all waits are bounded: on expiry the block records GVA_ERR_TIMEOUT, drains its copies and exits.
#pragma once

#include <cuda.h>

#include "gva_common.cuh"

namespace gva {

// ---- host-side state: the driver entry point for tensor-map encoding ---------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// Tensor maps depend only on the pools' addresses and sizes: they are encoded once per (pools, kernel kind) and kept in
// the handle, so a call in steady state pays no driver call for them.
struct alignas(64) MapPair {
    CUtensorMap tm_v, tm_k;
};
constexpr int kMaxDevicesCached = 64;
struct MmaHostState {
    EncodeTiledFn encode;
    int device;                      // the handle's device
    bool dry;                        // true: check support, set attributes and encode maps, but launch nothing
    static constexpr int kMaps = 8;
    struct Key {
        const void *v, *k;
        int num_pages, kind;
    } keys[kMaps];
    MapPair maps[kMaps];
    int n_maps, next_map;
    const MapPair *find(const void *v, const void *k, int num_pages, int kind) const {
        for (int i = 0; i < n_maps; ++i)
            if (keys[i].v == v && keys[i].k == k && keys[i].num_pages == num_pages && keys[i].kind == kind) return &maps[i];
        return nullptr;
    }
    MapPair *slot_for(const void *v, const void *k, int num_pages, int kind) {      // oldest entry is replaced
        const int i = n_maps < kMaps ? n_maps++ : (next_map++ % kMaps);
        keys[i] = Key{v, k, num_pages, kind};
        return &maps[i];
    }
    void forget_last() { if (n_maps > 0) keys[n_maps < kMaps ? --n_maps : ((next_map - 1) % kMaps)].v = nullptr; }
};

inline int mma_host_init(MmaHostState *st, int device) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
        return GVA_ERR_CUDA;
    st->encode = reinterpret_cast<EncodeTiledFn>(fn);
    st->dry = false;
    st->device = device;
    st->n_maps = 0;
    st->next_map = 0;
    return GVA_OK;
}

// ---- PTX wrappers ----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about kWaitLimitNs of wall time or when another thread of the block
// has aborted; never spins without limit.
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;
constexpr int kDrainPolls = 1 << 16;
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 127u) == 127u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) return false;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// The decode kernels read every cache byte exactly once per call: their loads carry an evict-first L2 policy, so the
// stream does not push the small things every call needs again (lengths, block table, queries, partial records, the
// kernels' own instructions) out of L2.
#ifndef GVA_STREAM_EVICT_FIRST
#define GVA_STREAM_EVICT_FIRST 1   // build-time knob: 0 = default L2 policy for the cache stream
#endif
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d_stream(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar, uint64_t pol) {
#if GVA_STREAM_EVICT_FIRST
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;\n" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar), "l"(pol)
        : "memory");
#else
    tma_load_2d(dst, map, x, y, bar);
#endif
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_k8(float (&c)[4], const uint32_t (&a)[2], uint32_t b0) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(b0));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
    return y;
}
// x = hi + lo with hi, lo bf16; returns hi in the low half-word, lo in the high half-word.
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    const __nv_bfloat16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
    return (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
}

// ---- compile-time geometry -------------------------------------------------------------------------
template <int DV, int DR, int TILE, bool GQA>
struct MmaTraits {
    static constexpr int BOXES = DV / 64;                       // 64-dim (128-byte) boxes per value row
    static constexpr int VBOX_BYTES = TILE * 128;               // one box of one group
    static constexpr int VTILE_BYTES = BOXES * VBOX_BYTES;      // one group's tile
    static constexpr int KR_ROW = DR * 2;                       // 32, 48 or 64 bytes
    static constexpr int KR_BYTES = TILE * KR_ROW;
    static constexpr int KSTEPS_V = DV / 16;
    static constexpr int KSTEPS_R = GQA ? 0 : DR / 16;          // full 16-wide k-steps over the RoPE dims
    static constexpr bool KREM8 = !GQA && (DR % 16) == 8;       // d_r = 24: one more 8-wide k-step (m16n8k8)
    static constexpr int KSTEPS = KSTEPS_V + KSTEPS_R;
    static constexpr int MT = DV / 16;                          // output m-tiles
    static constexpr int CHUNKS = TILE / 16;
    static constexpr int DQ = GQA ? DV : DV + DR;
    __host__ __device__ static constexpr int stage_bytes(int G) {
        return GQA ? 2 * G * VTILE_BYTES : G * VTILE_BYTES + ((KR_BYTES + 1023) & ~1023);
    }
    __host__ __device__ static constexpr int tail_bytes(int B, int nstage) {
        return nstage * 16 /* barriers */ + nstage * 16 /* per-stage meta */ + 16 /* abort */ + (B + 1) * 4;
    }
};

// Byte offset of 16-byte chunk `chunk` of row `row` inside a 128-byte-swizzled box (rows of 128 bytes).
__device__ __forceinline__ uint32_t swz128(int row, int chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }
// Positional-key tile: 32-byte rows use the 32-byte swizzle, 64-byte rows the 64-byte swizzle.
template <int KR_ROW>
__device__ __forceinline__ uint32_t swz_kr(int row, int chunk) {
    if constexpr (KR_ROW == 32) return row * 32 + ((chunk ^ ((row >> 2) & 1)) << 4);
    else return row * 64 + ((chunk ^ ((row >> 1) & 3)) << 4);
}

// {hi, lo} of x as two bf16 numbers with x ~= hi + lo: hi in the low half-word, lo in the high one.
// Four instructions: round, widen, subtract, round both.
__device__ __forceinline__ uint32_t split_hi_lo_fast(float x) {
    uint32_t t, d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(t) : "f"(0.f), "f"(x));          // low half = bf16(x)
    const float lo = x - __uint_as_float(t << 16);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(d) : "f"(lo), "f"(x));           // {bf16(lo), bf16(x)}
    return d;
}

// ---- what a thread block works on ------------------------------------------------------------------------
struct BlockWork {
    UnitPlan plan;
    BlockRange rg;        // first range of tiles (balanced: the head of the block's own range; uniform: its split)
    int first_unit;       // balanced: unit id of that range, -1 if the block has none
    int n_tickets;        // balanced: tail units on offer to whoever asks first
    bool uniform;
};

#ifndef GVA_MMA_DYNAMIC_TAIL
#define GVA_MMA_DYNAMIC_TAIL 1   // build-time knob: 0 = equal static ranges only
#endif
// Tail stealing pays where two or more blocks share an SM and their speeds differ by +-20 % (d_v = 64: measured -2.7 us
// of 100 on the long-context workload); with one block per SM (d_v = 128) speeds differ by +-4 % and the extra
// partial records cost more than the balance gains (measured +3.9 us of 180), so there the ranges stay static.
template <int DV>
__device__ __forceinline__ BlockWork decode_block_work(const DecodeParams &p, const int *s_off) {
    BlockWork w;
    w.uniform = p.num_splits > 0;
    w.plan = make_unit_plan(s_off[p.B], gridDim.x, GVA_MMA_DYNAMIC_TAIL != 0 && DV == 64);
    w.rg.lo = w.rg.hi = 0;
    w.rg.rec_fixed = -1;
    w.rg.b_first = 0;
    w.first_unit = -1;
    if (w.uniform) {
        w.rg = block_range(p, s_off);
    } else if ((int)blockIdx.x < w.plan.n_ranges) {
        w.first_unit = blockIdx.x * (w.plan.U + 1);          // the head of this block's own range
        unit_range(w.plan, blockIdx.x, 0, w.rg.lo, w.rg.hi);
        w.rg.b_first = (w.rg.lo < w.rg.hi) ? seq_of_tile(s_off, p.B, w.rg.lo) : 0;
    }
    w.n_tickets = w.uniform ? 0 : w.plan.n_ranges * w.plan.U;
    return w;
}

// Per-stage message from the producer to the consumers.
struct StageMeta {
    int n_valid;   // live tokens in the tile; -1 = no more tiles for this block
    int b;         // sequence
    int rec;       // partial record this tile's segment belongs to (before the per-warp multiplier)
    int flags;     // bit 0: first tile of its segment, bit 1: last tile of its segment; bits 8..: see QL > 1
};

// The producer lane of a tensor-core decode block: walks the block's tiles (its own range, then the tail units it
// wins), and for each one resolves the page, waits (bounded) for the ring slot, posts the stage message and calls
// issue(stage, page, first slot, full barrier), which posts the expected byte count and starts the copies.
// Early start (p.early_start, only behind step_front_kernel): nothing that kernel writes is touched before
// grid_dependency_wait() -- the tile that receives the token being appended is loaded only after the wait, and so is
// the ticket, which belongs to the previous call until then.
template <int TILE, int NSTAGE, bool MULTI, class Issue>
__device__ __forceinline__ void decode_producer(const DecodeParams &p, const BlockWork &w, const int *s_off, uint64_t *full_bar,
                                                uint64_t *empty_bar, StageMeta *s_meta, volatile int *s_abort, int ql,
                                                Issue issue) {
    bool waited = p.early_start == 0;
    bool ok = true;
    int issued = 0;       // tiles issued by this block: ring position
    int lo = w.rg.lo, hi = w.rg.hi, unit = w.first_unit;
    int b = w.rg.b_first;
    int32_t *ticket_ctr = p.sync + kSyncTicket + (p.epoch & 1);
    for (;;) {
        // the next tail unit is requested while this one is being issued
        int ticket = -1;
        bool asked = w.n_tickets == 0;
        for (int f = lo; f < hi && ok; ++f) {
            const int st = issued % NSTAGE;
            if (!waited && issued >= NSTAGE) {   // the ring is full: nothing more to gain from running ahead
                grid_dependency_wait();
                waited = true;
            }
            if (!asked && waited && hi - f <= 2) {   // late, so that tails go to whoever really is ahead
                ticket = atomicAdd(ticket_ctr, 1);
                asked = true;
            }
            while (f >= s_off[b + 1]) ++b;
            const int t0 = (f - s_off[b]) * TILE;
            const int pj = t0 / p.P, slot0 = t0 % p.P;
            // the three lookups are independent: request them together, use them afterwards
            const int len = p.seq_lens[b];
            const int ap = waited ? -1 : p.append_pos[b];
            long long page = p.block_table ? (long long)p.block_table[(size_t)b * p.max_pages + pj]
                                           : (long long)b * p.max_pages + pj;
            if (!waited && ap >= t0 && ap < t0 + TILE) {   // this tile receives the new token: it must be complete first
                grid_dependency_wait();
                waited = true;
            }
            int n_valid = min(TILE, len - t0);
            if (page < 0 || page >= p.num_pages) {
                report_error(p.dev_status, GVA_ERR_BAD_PAGE, b);
                page = 0;
                n_valid = 0;
            }
            // the bookkeeping above overlaps with the wait for the stage to be released
            if (!mbar_wait_bounded(smem_u32(&empty_bar[st]), ((issued / NSTAGE) & 1) ^ 1, s_abort)) {
                if (!*s_abort) report_error(p.dev_status, GVA_ERR_TIMEOUT, b);
                *s_abort = 1;
                ok = false;
                break;
            }
            StageMeta m;
            m.n_valid = n_valid;
            m.b = b;
            m.rec = w.uniform ? w.rg.rec_fixed : unit + b;
            m.flags = ((f == lo || f == s_off[b]) ? 1 : 0) | ((f + 1 == hi || f + 1 >= s_off[b + 1]) ? 2 : 0);
            if constexpr (MULTI) m.flags |= min(max(len - t0 - TILE, 0), ql - 1) << 8;   // tokens of the sequence beyond this tile, capped
            s_meta[st] = m;
            issue(st, page, slot0, smem_u32(&full_bar[st]));
            ++issued;
        }
        if (!ok) break;
        if (!asked) {
            if (!waited) {
                grid_dependency_wait();
                waited = true;
            }
            ticket = atomicAdd(ticket_ctr, 1);
        }
        if (ticket < 0 || ticket >= w.n_tickets) break;
        // ticket t -> tail j = 1 + t / n_ranges of range t % n_ranges: first every range's first tail, then the second, ...
        const int c = ticket % w.plan.n_ranges, j = 1 + ticket / w.plan.n_ranges;
        unit = c * (w.plan.U + 1) + j;
        unit_range(w.plan, c, j, lo, hi);
        if (lo < hi) b = seq_of_tile(s_off, p.B, lo);
    }
    if (ok) {
        // tell the consumers that nothing more is coming
        const int st = issued % NSTAGE;
        if (mbar_wait_bounded(smem_u32(&empty_bar[st]), ((issued / NSTAGE) & 1) ^ 1, s_abort)) {
            s_meta[st].n_valid = -1;
            mbar_arrive(smem_u32(&full_bar[st]));
        } else {
            if (!*s_abort) report_error(p.dev_status, GVA_ERR_TIMEOUT, b);
            *s_abort = 1;
            ok = false;
        }
    }
    if (!ok) {
        // drain: every copy this block started must land before its shared memory is released
        const int first = max(0, issued - NSTAGE);
        for (int i = first; i < issued; ++i) {
            const int st = i % NSTAGE;
            for (int it = 0; it < kDrainPolls; ++it)
                if (mbar_try_wait(smem_u32(&full_bar[st]), (i / NSTAGE) & 1)) break;
        }
    }
}

// QL > 1 (multi-token decode, QL = 2 or 4 new tokens per sequence): the 4 heads x QL tokens of a group are the N
// columns, 8 per N-block, column c = slot * 4 + head with slot the token's index among the new ones; the queries and
// the weights go in as plain bf16 (the hi/lo halves of the single-token layout have become the second token), slot s
// attends to seq_len - (q_len - 1 - s) tokens, and the partial records and outputs use q_len * H pseudo-heads, slot * H + head.
// CW > 1: the columns of a group are split over CW consumer warps, warp cw taking slots cw * QL .. cw * QL + QL - 1 of
// the same shared-memory tile (QL = 4, CW = 2: up to eight new tokens per sequence; one such block fills an SM).
// With DecodeParams::cu_q every sequence has its own number of new tokens (at most q_len, possibly none).
template <int DV, int DR, int TILE, int NSTAGE, int WPG, bool GQA, int QL = 1, int CW = 1>
__global__ void __launch_bounds__(32 * 9)
decode_mma_kernel(DecodeParams p, const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_k) {
    using T = MmaTraits<DV, DR, TILE, GQA>;
    constexpr int CPW = T::CHUNKS / WPG;          // 16-token chunks per consumer warp and tile
    static_assert(CPW >= 1 && CPW * WPG == T::CHUNKS, "tile must split evenly over the group's warps");
    grid_dependency_launch();
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // dynamic shared memory is only guaranteed 16-byte aligned: round up to the swizzle atom
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    static_assert(QL == 1 || ((QL == 2 || QL == 4) && !GQA && (DR % 8) == 0), "multi-token decode: 2 or 4 new tokens per warp, GVA cache, d_r a multiple of 8");
    constexpr int NBK = QL == 1 ? 1 : QL / 2;     // N-blocks of 8 columns
    const int G = p.G, H = p.H;
    static_assert(CW == 1 || (QL > 1 && WPG == 1), "column-split warps belong to the multi-token kernel");
    const int ql = QL == 1 ? 1 : p.q_len;         // new tokens per sequence (<= QL * CW; slots beyond it stay empty)
    const int HQ = H * ql;                        // pseudo-heads of the partial records
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n_consumers = G * WPG * CW;
    const int stage_bytes = T::stage_bytes(G);

    unsigned char *tail = smem + (size_t)NSTAGE * stage_bytes;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(tail);
    uint64_t *empty_bar = full_bar + NSTAGE;
    StageMeta *s_meta = reinterpret_cast<StageMeta *>(empty_bar + NSTAGE);
    volatile int *s_abort = reinterpret_cast<volatile int *>(s_meta + NSTAGE);
    int *s_off = reinterpret_cast<int *>(s_meta + NSTAGE) + 4;

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), n_consumers);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        // fetch the two tensor-map descriptors now, not at the first copy
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
    }
    // Early start (only behind step_front_kernel, which has already waited for everything before it): the
    // tile bookkeeping and the producer's first loads run while the front kernel computes.  Nothing the front
    // kernel writes is touched before grid_dependency_wait(): consumers wait before reading the absorbed
    // query, the producer waits before loading the tile that holds the token being appended, and the
    // workspace is written only after the wait.
    const bool early = p.early_start != 0;
    if (tid == 0) {
        trace(kTrDecodeEnterMin, p.epoch);
        trace(kTrDecodeEnterMax, p.epoch);
    }
    if (!early) grid_dependency_wait();
    compute_tile_offsets<TILE>(p, s_off);   // ends with __syncthreads(): barriers are initialised for everyone
    const BlockWork w = decode_block_work<DV>(p, s_off);
    const UnitPlan &plan = w.plan;
    const BlockRange &rg = w.rg;
    if (w.uniform ? rg.hi <= rg.lo : (w.first_unit < 0 && w.n_tickets == 0)) {
        // nothing to stream.  Uniform mode: an empty split still owns its records (weight 0 in the merge); balanced
        // mode: more blocks than ranges and no tails to share.
        if (early) grid_dependency_wait();
        block0_duties(p, s_off, plan, tid, blockDim.x);
        if (w.uniform)
            for (int i = tid; i < HQ * WPG; i += blockDim.x) {
                p.rec_ml[((size_t)rg.rec_fixed * WPG * HQ + i) * 2] = -INFINITY;
                p.rec_ml[((size_t)rg.rec_fixed * WPG * HQ + i) * 2 + 1] = 0.f;
            }
        return;
    }

    if (warp == n_consumers) {
        // ================================ producer (one elected lane) ================================
        if (lane == 0) {
            const uint64_t pol = l2_policy_evict_first();
            decode_producer<TILE, NSTAGE, (QL > 1)>(p, w, s_off, full_bar, empty_bar, s_meta, s_abort, ql,
                [&](int st, long long page, int slot0, uint32_t bar) {
                    const uint32_t base = smem_u32(smem + (size_t)st * stage_bytes);
                    mbar_expect_tx(bar, GQA ? 2 * G * T::VTILE_BYTES : G * T::VTILE_BYTES + T::KR_BYTES);
                    if constexpr (!GQA && DR > 0) tma_load_2d_stream(base + G * T::VTILE_BYTES, &tm_k, 0, (int)(page * p.P + slot0), bar, pol);
                    for (int g = 0; g < G; ++g) {
                        const int row = (int)((page * G + g) * p.P + slot0);
                        if constexpr (GQA) {
#pragma unroll
                            for (int bx = 0; bx < T::BOXES; ++bx)
                                tma_load_2d_stream(base + (G + g) * T::VTILE_BYTES + bx * T::VBOX_BYTES, &tm_k, bx * 64, row, bar, pol);
                        }
#pragma unroll
                        for (int bx = 0; bx < T::BOXES; ++bx)
                            tma_load_2d_stream(base + g * T::VTILE_BYTES + bx * T::VBOX_BYTES, &tm_v, bx * 64, row, bar, pol);
                    }
                });
        }
    } else {
        // ============ consumer: value group g, token chunks [part*CPW, part*CPW + CPW) of every tile ============
        const int g = warp / (WPG * CW);
        const int part = (warp / CW) % WPG;
        const int slot_base = (warp % CW) * QL;      // multi-token decode: first new-token slot of this warp's columns
        const int jh = lane & 3;          // head within the group this lane's score/output columns belong to
        const int r8 = lane >> 2;         // row within an 8-row block
        // ldmatrix lane addressing inside a 16-token chunk of a 128-byte-swizzled box.  The 16-byte chunk index
        // is (k-step or m-tile) * 2 + hi, XOR row % 8; the compile-time part is applied as "^ (idx << 5)" below.
        const int r7 = lane & 7;
        const int row_qk = r7 + ((lane >> 3) & 1) * 8, hi_qk = lane >> 4;          // matrices: (r0-7,k0-7) (r8-15,k0-7) (r0-7,k8-15) (r8-15,k8-15)
        const int row_pv = r7 + (lane >> 4) * 8, hi_pv = (lane >> 3) & 1;          // transposed: (t0-7,d0-7) (t0-7,d8-15) (t8-15,d0-7) (t8-15,d8-15)
        const uint32_t off_qk = row_qk * 128 + ((hi_qk ^ r7) << 4);
        const uint32_t off_pv = row_pv * 128 + ((hi_pv ^ r7) << 4);
        // positional-key tile: 32-byte rows carry the 32-byte swizzle, 64-byte rows the 64-byte one; 48-byte rows
        // (d_r = 24) are unswizzled -- a 48-byte stride is conflict-free for ldmatrix as it is
        const uint32_t off_kr = (T::KR_ROW == 32)   ? row_qk * 32 + ((hi_qk ^ ((row_qk >> 2) & 1)) << 4)
                                : (T::KR_ROW == 64) ? row_qk * 64 + ((hi_qk ^ ((row_qk >> 1) & 3)) << 4)
                                                    : row_qk * 48 + (hi_qk << 4);
        if constexpr (QL == 1) {
        uint32_t qf[T::KSTEPS][2];        // B fragments of Q^T: column n = lane/4 = 2*head + {hi, lo}
        uint32_t qf8 = 0;                 // d_r = 24: B fragment of the last 8 RoPE dims
        float oacc[T::MT][4];
        float m_run = -INFINITY, l_run = 0.f;
        const float scale = p.scale_log2;
        const int lo_part = r8 & 1;

        // absorbed query of head (lane/4)/2, hi or lo part by (lane/4)&1, as mma B fragments
        auto load_query = [&](int b) {
            const float *q = p.q + ((size_t)b * H + g * kHeadsPerGroup + (r8 >> 1)) * T::DQ;
#pragma unroll
            for (int kk = 0; kk < T::KSTEPS; ++kk) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const float2 v = *reinterpret_cast<const float2 *>(q + kk * 16 + half * 8 + 2 * jh);
                    const uint32_t sx = split_hi_lo(v.x), sy = split_hi_lo(v.y);
                    qf[kk][half] = lo_part ? ((sx >> 16) | (sy & 0xffff0000u)) : ((sx & 0xffffu) | (sy << 16));
                }
            }
            if constexpr (T::KREM8) {
                const float2 v = *reinterpret_cast<const float2 *>(q + T::KSTEPS * 16 + 2 * jh);
                const uint32_t sx = split_hi_lo(v.x), sy = split_hi_lo(v.y);
                qf8 = lo_part ? ((sx >> 16) | (sy & 0xffff0000u)) : ((sx & 0xffffu) | (sy << 16));
            }
        };
        if (early) grid_dependency_wait();
        block0_duties(p, s_off, plan, tid, n_consumers * 32);
        // the first sequence is known before any tile arrives: fetch its query while the first copies fly
        int cur_b = -1;
        if (rg.lo < rg.hi) {
            cur_b = rg.b_first;
            load_query(cur_b);
        }

#pragma unroll 1
        for (int i = 0;; ++i) {
            const int st = i % NSTAGE;
            if (!mbar_wait_bounded(smem_u32(&full_bar[st]), (i / NSTAGE) & 1, s_abort)) {
                if (!*s_abort && lane == 0) report_error(p.dev_status, GVA_ERR_TIMEOUT, cur_b < 0 ? 0 : cur_b);
                *s_abort = 1;
                break;
            }
            const StageMeta meta = s_meta[st];
            const int n_valid = meta.n_valid;
            if (n_valid < 0) break;       // producer is done
            if (i == 0 && tid == 0) {
                trace(kTrFirstTileMin, p.epoch);
                trace(kTrFirstTileMax, p.epoch);
            }
            const int b = meta.b;
            if (meta.flags & 1) {         // a new segment: its own softmax state (and query, if the sequence changed)
                if (b != cur_b) {
                    cur_b = b;
                    load_query(b);
                }
                m_run = -INFINITY;
                l_run = 0.f;
#pragma unroll
                for (int mt = 0; mt < T::MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) oacc[mt][e] = 0.f;
            }
            unsigned char *stage = smem + (size_t)st * stage_bytes;
            unsigned char *vt = stage + (size_t)g * T::VTILE_BYTES;
            const int row0 = part * CPW * 16;                 // first token row of this warp's share of the tile
            const bool ragged = n_valid < row0 + CPW * 16;
            if (ragged) {
                // rows past the sequence end may hold anything (NaN included): zero this warp's share of them
                // so that a zero weight times such a row stays zero
                const int z0 = max(n_valid, row0);
                const int n_zero_chunks = (row0 + CPW * 16 - z0) * 8;
                for (int c = lane; c < n_zero_chunks * T::BOXES; c += 32) {
                    const int bx = c / n_zero_chunks, cc = c % n_zero_chunks;
                    *reinterpret_cast<uint4 *>(vt + bx * T::VBOX_BYTES + (z0 + cc / 8) * 128 + (cc % 8) * 16) =
                        make_uint4(0, 0, 0, 0);
                }
                // generic-proxy writes must be ordered before the TMA write that later refills the stage
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                __syncwarp();
            }
            const uint32_t vt_u32 = smem_u32(vt) + row0 * 128;
            const uint32_t ks_u32 = GQA ? smem_u32(stage + (size_t)(G + g) * T::VTILE_BYTES) + row0 * 128 : vt_u32;
            const uint32_t kr_u32 = smem_u32(stage + (size_t)G * T::VTILE_BYTES) + row0 * T::KR_ROW;

            // ---- S^T = (score source tile) . Q^T, 16 tokens per m-tile ----
            float sacc[CPW][4];
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sacc[c][e] = 0.f;
#pragma unroll
                for (int kk = 0; kk < T::KSTEPS_V; ++kk) {
                    uint32_t a[4];
                    ldsm_x4(ks_u32 + (kk >> 2) * T::VBOX_BYTES + c * 2048 + (off_qk ^ ((kk & 3) << 5)), a);
                    mma_bf16(sacc[c], a, qf[kk][0], qf[kk][1]);
                }
                if constexpr (!GQA) {
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS_R; ++kk) {
                        uint32_t a[4];
                        ldsm_x4(kr_u32 + c * 16 * T::KR_ROW + (off_kr ^ (kk << 5)), a);
                        mma_bf16(sacc[c], a, qf[T::KSTEPS_V + kk][0], qf[T::KSTEPS_V + kk][1]);
                    }
                    if constexpr (T::KREM8) {     // dims 16..23: rows 0-7 and 8-15, third 16-byte chunk of each row
                        uint32_t a2[2];
                        ldsm_x2(kr_u32 + c * 16 * T::KR_ROW + row_qk * T::KR_ROW + 32, a2);
                        mma_bf16_k8(sacc[c], a2, qf8);
                    }
                }
            }
            // ---- online softmax for head jh over this warp's tokens (rows r8, r8+8 of every m-tile) ----
            float sr[CPW][2];              // raw scores (hi + lo columns summed)
            float tmax = -INFINITY;
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                sr[c][0] = sacc[c][0] + sacc[c][1];
                sr[c][1] = sacc[c][2] + sacc[c][3];
                if (ragged) {
                    const int t_lo = row0 + c * 16 + r8;
                    if (t_lo >= n_valid) sr[c][0] = -INFINITY;
                    if (t_lo + 8 >= n_valid) sr[c][1] = -INFINITY;
                }
                tmax = fmaxf(tmax, fmaxf(sr[c][0], sr[c][1]));
            }
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 8));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
            const float m_new = fmaxf(m_run, tmax * scale);          // scale > 0: max commutes with it
            const bool live = m_new != -INFINITY;
            const float m_use = live ? m_new : 0.f;                  // keeps (-inf) - (-inf) out of the exponent
            const float corr = fast_exp2(m_run - m_use);             // 2^(-inf) = 0 for the first live tile
            m_run = m_new;
            l_run *= corr;
#pragma unroll
            for (int mt = 0; mt < T::MT; ++mt)
#pragma unroll
                for (int e = 0; e < 4; ++e) oacc[mt][e] *= corr;

            // ---- O^T += V_tile^T . P^T ----
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                const float p0 = fast_exp2(fmaf(sr[c][0], scale, -m_use));
                const float p1 = fast_exp2(fmaf(sr[c][1], scale, -m_use));
                l_run += p0 + p1;
                // (hi, lo) of p for token row r8 / r8+8 and columns 2*jh, 2*jh+1 -> transpose to B fragments
                const uint32_t pb0 = movmatrix_trans(split_hi_lo_fast(p0));
                const uint32_t pb1 = movmatrix_trans(split_hi_lo_fast(p1));
#pragma unroll
                for (int mt = 0; mt < T::MT; ++mt) {
                    uint32_t a[4];
                    ldsm_x4_trans(vt_u32 + (mt >> 2) * T::VBOX_BYTES + c * 2048 + (off_pv ^ ((mt & 3) << 5)), a);
                    mma_bf16(oacc[mt], a, pb0, pb1);
                }
            }
            // release the stage to the producer
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&empty_bar[st]));

            // ---- segment end: write this (unit, sequence, part) partial ----
            if (meta.flags & 2) {
                const int rec = meta.rec * WPG + part;
                float l = l_run;
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                const size_t rh = (size_t)rec * H + g * kHeadsPerGroup + jh;
                float *o_dst = p.rec_o + rh * DV;
#pragma unroll
                for (int mt = 0; mt < T::MT; ++mt) {
                    o_dst[mt * 16 + r8] = oacc[mt][0] + oacc[mt][1];
                    o_dst[mt * 16 + r8 + 8] = oacc[mt][2] + oacc[mt][3];
                }
                if (r8 == 0) {
                    p.rec_ml[rh * 2] = m_run;
                    p.rec_ml[rh * 2 + 1] = l;
                }
            }
        }

        } else {
            // ================= multi-token decode: QL new tokens per sequence, columns = slot * 4 + head =================
            // B fragments of Q^T: column n = lane / 4 of N-block nb.  The f32 query goes in as two bf16 numbers, q = hi + lo, and
            // the score product is taken with both (twice the score MMAs): with hi alone a score s is off by about |s| 2^-9,
            // which on sharply peaked rows is what limits the accuracy of the output.
            uint32_t qf[T::KSTEPS][NBK][2], qlo[T::KSTEPS][NBK][2];
            uint32_t qf8[NBK], qlo8[NBK];          // d_r = 24: B fragments of the last 8 RoPE dims
            float oacc[T::MT][NBK][4];
            float m_run[NBK][2], l_run[NBK][2];   // per column of this lane: columns 2 jh, 2 jh + 1 of every N-block
            const float scale = p.scale_log2;
            // the lane's B-fragment column n = lane / 4 = r8 is (slot 2 nb + n / 4, head n % 4)
            int cur_ql = ql;                       // new tokens of the current sequence
            auto load_query = [&](int b) {
                size_t row0 = (size_t)b * ql;
                cur_ql = ql;
                if (p.cu_q) {                      // its own count and first query row per sequence
                    const int r_lo = p.cu_q[b];
                    row0 = (size_t)r_lo;
                    cur_ql = min(max(p.cu_q[b + 1] - r_lo, 0), ql);
                }
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb) {
                    const int slot = slot_base + 2 * nb + (r8 >> 2), head = r8 & 3;
                    const bool present = slot < cur_ql;   // an absent slot gets a zero query; its columns are masked everywhere
                    const float *q = p.q + ((row0 + (present ? slot : 0)) * H + g * kHeadsPerGroup + head) * T::DQ;
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS; ++kk)
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            float2 v = make_float2(0.f, 0.f);
                            if (present) v = *reinterpret_cast<const float2 *>(q + kk * 16 + half * 8 + 2 * jh);
                            uint32_t w, wl;
                            asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(w) : "f"(v.y), "f"(v.x));
                            asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(wl) : "f"(v.y - __uint_as_float(w & 0xffff0000u)), "f"(v.x - __uint_as_float(w << 16)));
                            qf[kk][nb][half] = w;
                            qlo[kk][nb][half] = wl;
                        }
                    qf8[nb] = qlo8[nb] = 0;
                    if constexpr (T::KREM8) {
                        float2 v = make_float2(0.f, 0.f);
                        if (present) v = *reinterpret_cast<const float2 *>(q + T::KSTEPS * 16 + 2 * jh);
                        uint32_t w, wl;
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(w) : "f"(v.y), "f"(v.x));
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(wl) : "f"(v.y - __uint_as_float(w & 0xffff0000u)), "f"(v.x - __uint_as_float(w << 16)));
                        qf8[nb] = w;
                        qlo8[nb] = wl;
                    }
                }
            };
            if (early) grid_dependency_wait();
            block0_duties(p, s_off, plan, tid, n_consumers * 32);
            int cur_b = -1;
            if (rg.lo < rg.hi) {
                cur_b = rg.b_first;
                load_query(cur_b);
            }
#pragma unroll 1
            for (int i = 0;; ++i) {
                const int st = i % NSTAGE;
                if (!mbar_wait_bounded(smem_u32(&full_bar[st]), (i / NSTAGE) & 1, s_abort)) {
                    if (!*s_abort && lane == 0) report_error(p.dev_status, GVA_ERR_TIMEOUT, cur_b < 0 ? 0 : cur_b);
                    *s_abort = 1;
                    break;
                }
                const StageMeta meta = s_meta[st];
                const int n_valid = meta.n_valid;
                if (n_valid < 0) break;       // producer is done
                const int b = meta.b;
                if (meta.flags & 1) {         // a new segment: its own softmax state (and queries, if the sequence changed)
                    if (b != cur_b) {
                        cur_b = b;
                        load_query(b);
                    }
#pragma unroll
                    for (int nb = 0; nb < NBK; ++nb) {
                        m_run[nb][0] = m_run[nb][1] = -INFINITY;
                        l_run[nb][0] = l_run[nb][1] = 0.f;
#pragma unroll
                        for (int mt = 0; mt < T::MT; ++mt)
#pragma unroll
                            for (int e = 0; e < 4; ++e) oacc[mt][nb][e] = 0.f;
                    }
                }
                unsigned char *stage = smem + (size_t)st * stage_bytes;
                unsigned char *vt = stage + (size_t)g * T::VTILE_BYTES;
                const int row0 = part * CPW * 16;
                // tokens of this tile that slot s may see: n_valid + (tokens of the sequence beyond the tile, capped) - (QL - 1 - s)
                const int reach = n_valid + min((meta.flags >> 8) & 0xff, max(cur_ql - 1, 0)) - (cur_ql - 1);
                const bool ragged = n_valid < row0 + CPW * 16;
                if (ragged) {
                    const int z0 = max(n_valid, row0);
                    const int n_zero_chunks = (row0 + CPW * 16 - z0) * 8;
                    for (int c = lane; c < n_zero_chunks * T::BOXES; c += 32) {
                        const int bx = c / n_zero_chunks, cc = c % n_zero_chunks;
                        *reinterpret_cast<uint4 *>(vt + bx * T::VBOX_BYTES + (z0 + cc / 8) * 128 + (cc % 8) * 16) =
                            make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    __syncwarp();
                }
                const bool masked = reach < row0 + CPW * 16 || cur_ql < slot_base + QL;      // some slot does not see the whole share of this warp
                const uint32_t vt_u32 = smem_u32(vt) + row0 * 128;
                const uint32_t kr_u32 = smem_u32(stage + (size_t)G * T::VTILE_BYTES) + row0 * T::KR_ROW;

                // ---- S^T = V_tile . Q^T (+ positional part): 16 tokens per m-tile, 8 columns per N-block ----
                float sacc[CPW][NBK][4];
#pragma unroll
                for (int c = 0; c < CPW; ++c) {
#pragma unroll
                    for (int nb = 0; nb < NBK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) sacc[c][nb][e] = 0.f;
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS_V; ++kk) {
                        uint32_t a[4];
                        ldsm_x4(vt_u32 + (kk >> 2) * T::VBOX_BYTES + c * 2048 + (off_qk ^ ((kk & 3) << 5)), a);
#pragma unroll
                        for (int nb = 0; nb < NBK; ++nb) {
                            mma_bf16(sacc[c][nb], a, qlo[kk][nb][0], qlo[kk][nb][1]);
                            mma_bf16(sacc[c][nb], a, qf[kk][nb][0], qf[kk][nb][1]);
                        }
                    }
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS_R; ++kk) {
                        uint32_t a[4];
                        ldsm_x4(kr_u32 + c * 16 * T::KR_ROW + (off_kr ^ (kk << 5)), a);
#pragma unroll
                        for (int nb = 0; nb < NBK; ++nb) {
                            mma_bf16(sacc[c][nb], a, qlo[T::KSTEPS_V + kk][nb][0], qlo[T::KSTEPS_V + kk][nb][1]);
                            mma_bf16(sacc[c][nb], a, qf[T::KSTEPS_V + kk][nb][0], qf[T::KSTEPS_V + kk][nb][1]);
                        }
                    }
                    if constexpr (T::KREM8) {     // dims 16..23: rows 0-7 and 8-15, third 16-byte chunk of each row
                        uint32_t a2[2];
                        ldsm_x2(kr_u32 + c * 16 * T::KR_ROW + row_qk * T::KR_ROW + 32, a2);
#pragma unroll
                        for (int nb = 0; nb < NBK; ++nb) {
                            mma_bf16_k8(sacc[c][nb], a2, qlo8[nb]);
                            mma_bf16_k8(sacc[c][nb], a2, qf8[nb]);
                        }
                    }
                }
                // ---- online softmax per column: this lane holds columns 2 jh, 2 jh + 1 of every N-block at token rows
                //      r8 and r8 + 8 of every m-tile; both columns belong to slot 2 nb + jh / 2 ----
                float corr[NBK][2], m_use[NBK][2];
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb) {
                    const int slot_l = slot_base + 2 * nb + (jh >> 1);
                    const int lim = slot_l < cur_ql ? reach + slot_l : 0;     // tokens of the tile this slot sees (an absent slot: none)
                    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < CPW; ++c) {
                        if (masked) {
                            const int t_lo = row0 + c * 16 + r8;
                            if (t_lo >= lim) sacc[c][nb][0] = sacc[c][nb][1] = -INFINITY;
                            if (t_lo + 8 >= lim) sacc[c][nb][2] = sacc[c][nb][3] = -INFINITY;
                        }
                        tmax[0] = fmaxf(tmax[0], fmaxf(sacc[c][nb][0], sacc[c][nb][2]));
                        tmax[1] = fmaxf(tmax[1], fmaxf(sacc[c][nb][1], sacc[c][nb][3]));
                    }
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        float t = tmax[e];
                        t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 4));
                        t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 8));
                        t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 16));
                        const float m_new = fmaxf(m_run[nb][e], t * scale);
                        m_use[nb][e] = (m_new != -INFINITY) ? m_new : 0.f;    // keeps (-inf) - (-inf) out of the exponent
                        corr[nb][e] = fast_exp2(m_run[nb][e] - m_use[nb][e]);
                        m_run[nb][e] = m_new;
                        l_run[nb][e] *= corr[nb][e];
                    }
#pragma unroll
                    for (int mt = 0; mt < T::MT; ++mt) {
                        oacc[mt][nb][0] *= corr[nb][0];
                        oacc[mt][nb][1] *= corr[nb][1];
                        oacc[mt][nb][2] *= corr[nb][0];
                        oacc[mt][nb][3] *= corr[nb][1];
                    }
                }
                // ---- O^T += V_tile^T . P^T ----
#pragma unroll
                for (int c = 0; c < CPW; ++c) {
                    uint32_t pb[NBK][2];
#pragma unroll
                    for (int nb = 0; nb < NBK; ++nb) {
                        const float p00 = fast_exp2(fmaf(sacc[c][nb][0], scale, -m_use[nb][0]));   // row r8,     column 2 jh
                        const float p01 = fast_exp2(fmaf(sacc[c][nb][1], scale, -m_use[nb][1]));   // row r8,     column 2 jh + 1
                        const float p10 = fast_exp2(fmaf(sacc[c][nb][2], scale, -m_use[nb][0]));   // row r8 + 8, column 2 jh
                        const float p11 = fast_exp2(fmaf(sacc[c][nb][3], scale, -m_use[nb][1]));
                        l_run[nb][0] += p00 + p10;
                        l_run[nb][1] += p01 + p11;
                        uint32_t w0, w1;
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(w0) : "f"(p01), "f"(p00));
                        asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(w1) : "f"(p11), "f"(p10));
                        pb[nb][0] = movmatrix_trans(w0);
                        pb[nb][1] = movmatrix_trans(w1);
                    }
#pragma unroll
                    for (int mt = 0; mt < T::MT; ++mt) {
                        uint32_t a[4];
                        ldsm_x4_trans(vt_u32 + (mt >> 2) * T::VBOX_BYTES + c * 2048 + (off_pv ^ ((mt & 3) << 5)), a);
#pragma unroll
                        for (int nb = 0; nb < NBK; ++nb) mma_bf16(oacc[mt][nb], a, pb[nb][0], pb[nb][1]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&empty_bar[st]));

                // ---- segment end: one partial per (unit, sequence, part) and pseudo-head slot * H + head ----
                if (meta.flags & 2) {
                    const int rec = meta.rec * WPG + part;
#pragma unroll
                    for (int nb = 0; nb < NBK; ++nb)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float l = l_run[nb][e];
                            l += __shfl_xor_sync(0xffffffffu, l, 4);
                            l += __shfl_xor_sync(0xffffffffu, l, 8);
                            l += __shfl_xor_sync(0xffffffffu, l, 16);
                            const int col = 2 * jh + e;                       // column of N-block nb: slot slot_base + 2 nb + col / 4, head col % 4
                            const int slot_w = slot_base + 2 * nb + (col >> 2);
                            if (slot_w >= cur_ql) continue;                    // (uniform over the lanes that reduce together)
                            const size_t rh = (size_t)rec * HQ + (size_t)slot_w * H + g * kHeadsPerGroup + (col & 3);
                            float *o_dst = p.rec_o + rh * DV;
#pragma unroll
                            for (int mt = 0; mt < T::MT; ++mt) {
                                o_dst[mt * 16 + r8] = oacc[mt][nb][e];
                                o_dst[mt * 16 + r8 + 8] = oacc[mt][nb][2 + e];
                            }
                            if (r8 == 0) {
                                p.rec_ml[rh * 2] = m_run[nb][e];
                                p.rec_ml[rh * 2 + 1] = l;
                            }
                        }
                }
            }
        }
    }
    // keep shared memory alive until every warp (and every copy in flight) is done
    __syncthreads();
    if (tid == 0) {
        trace(kTrDecodeExitMin, p.epoch);
        trace(kTrDecodeExitMax, p.epoch);
    }
}

// ---- host: support check, tensor maps, launch ------------------------------------------------------
// Tokens per tile: sized so that three stages of (G value tiles + the score-source tile(s)) fit in shared memory.
inline int mma_tile_for(const gva_config &cfg, bool gqa) {
    if (cfg.d_v == 64) return cfg.page_size % 64 == 0 ? 64 : 32;
    return gqa ? 16 : 32;
}
// Consumer warps per value group (each takes an equal share of a tile's 16-token chunks and writes its own partial).
#ifndef GVA_MMA_WPG64
#define GVA_MMA_WPG64 1   // build-time tuning knob for the d_v = 64 kernels: 1 or 2 (measured equal; 1 halves the partial records)
#endif
inline int mma_warps_per_group(const gva_config &cfg, bool /*gqa*/) { return cfg.d_v == 64 ? GVA_MMA_WPG64 : 1; }

inline bool mma_supported(const gva_config &cfg, bool gqa) {
    return cfg.cache_dtype == GVA_BF16 && cfg.page_size % mma_tile_for(cfg, gqa) == 0;
}

inline bool encode_map(const MmaHostState &st, CUtensorMap *map, const void *base, uint64_t inner, uint64_t rows,
                       uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz) {
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return st.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Resident blocks per SM that the grid of the 16-bit tensor-core kernel is sized for at most: what the shared memory
// of an SM holds of its three-stage rings, at most 4.  The workspace bound uses the same number.
inline int mma_blocks_per_sm_cap(const gva_config &cfg, bool gqa, int smem_per_sm) {
    const int tile = (cfg.d_v == 64) ? (cfg.page_size % 64 == 0 ? 64 : 32) : (gqa ? 16 : 32);
    const int vtile = (cfg.d_v / 64) * tile * 128;
    const int kr = (tile * cfg.d_r * 2 + 1023) & ~1023;
    const int stage = gqa ? 2 * cfg.G * vtile : cfg.G * vtile + (cfg.d_r > 0 ? kr : 0);
    const int per_block = 1024 + 3 * stage + 1024;      // alignment slack + rings + the per-block reservation of the hardware
    const int n = smem_per_sm / per_block;
    return n < 1 ? 1 : (n > 4 ? 4 : n);
}

template <int DV, int DR, int TILE, int NSTAGE, int WPG, bool GQA, int QL = 1, int CW = 1>
int launch_mma_t(const gva_config &cfg, MmaHostState &st, int sm_count, int smem_optin, const DecodeParams &p, int B,
                 int max_seq_len, int num_splits, int max_blocks, cudaStream_t stream, int *n_blocks_out) {
    using T = MmaTraits<DV, DR, TILE, GQA>;
    const int G = cfg.G;
    const size_t smem = 1024 + (size_t)NSTAGE * T::stage_bytes(G) + T::tail_bytes(B, NSTAGE) + 16;
    if (smem > (size_t)smem_optin) return GVA_ERR_UNSUPPORTED;
    auto fn = decode_mma_kernel<DV, DR, TILE, NSTAGE, WPG, GQA, QL, CW>;
    // the attribute and the occupancy figure are asked for once per (kernel, device, shared-memory size), not per call
    static int s_smem_set[kMaxDevicesCached] = {}, s_occupancy[kMaxDevicesCached] = {};
    const int dev = st.device >= 0 && st.device < kMaxDevicesCached ? st.device : 0;
    const int threads = 32 * (G * WPG * CW + 1);
    if (threads > 32 * 9) return GVA_ERR_UNSUPPORTED;
    if (s_smem_set[dev] != (int)smem || st.device >= kMaxDevicesCached) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GVA_ERR_CUDA;
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, smem) != cudaSuccess) return GVA_ERR_CUDA;
        s_occupancy[dev] = per_sm;
        s_smem_set[dev] = (int)smem;
    }
    const void *kptr = GQA ? p.k_pool : p.kr_pool;
    const MapPair *mp = st.find(p.v_pool, kptr, p.num_pages, GQA ? 1 : 0);
    if (!mp) {
        MapPair *m = st.slot_for(p.v_pool, kptr, p.num_pages, GQA ? 1 : 0);
        const uint64_t vrows = (uint64_t)p.num_pages * G * p.P;
        bool ok = encode_map(st, &m->tm_v, p.v_pool, DV, vrows, 64, TILE, CU_TENSOR_MAP_SWIZZLE_128B);
        if (ok && GQA) {
            ok = encode_map(st, &m->tm_k, p.k_pool, DV, vrows, 64, TILE, CU_TENSOR_MAP_SWIZZLE_128B);
        } else if (ok && DR == 0) {
            m->tm_k = m->tm_v;      // value-only cache: there is no positional-key tile to describe (the kernel never uses this map)
        } else if (ok) {
            ok = encode_map(st, &m->tm_k, p.kr_pool, DR, (uint64_t)p.num_pages * p.P, DR, TILE,
                            DR == 16   ? CU_TENSOR_MAP_SWIZZLE_32B
                            : DR == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                       : CU_TENSOR_MAP_SWIZZLE_NONE);
        }
        if (!ok) {
            st.forget_last();
            return GVA_ERR_CUDA;
        }
        mp = m;
    }
    int grid;
    if (num_splits > 0) {
        grid = B * num_splits;
    } else {
        int per_sm = s_occupancy[dev];
        per_sm = per_sm < 1 ? 1 : (per_sm > 4 ? 4 : per_sm);
        const long long tiles_ub = (long long)B * ((max_seq_len + TILE - 1) / TILE);
        long long want = (long long)per_sm * sm_count;
        if (want > max_blocks) want = max_blocks;      // never more blocks than the workspace was sized for
        grid = (int)(tiles_ub < want ? (tiles_ub < 1 ? 1 : tiles_ub) : want);
    }
    *n_blocks_out = grid;
    if (st.dry) return GVA_OK;
    DecodeParams pp = p;
    pp.rec_mult = WPG;
    if (launch_pdl(fn, dim3(grid), dim3(threads), smem, stream, pp, mp->tm_v, mp->tm_k) != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

template <bool GQA>
int launch_decode_mma(const gva_config &cfg, MmaHostState &st, int sm_count, int smem_optin, const DecodeParams &p,
                      int B, int max_seq_len, int num_splits, int max_blocks, cudaStream_t stream, int *n_blocks_out,
                      int *tile_out, int *rec_mult_out) {
    if (!mma_supported(cfg, GQA)) return GVA_ERR_UNSUPPORTED;
    // the tensor maps address rows with 32-bit coordinates
    if ((uint64_t)p.num_pages * cfg.G * cfg.page_size >= (1ull << 31)) return GVA_ERR_UNSUPPORTED;
    *tile_out = mma_tile_for(cfg, GQA);
    *rec_mult_out = mma_warps_per_group(cfg, GQA);
    if (cfg.d_v == 64 && cfg.d_r == 24 && !GQA) {
        if (*tile_out == 64)
            return launch_mma_t<64, 24, 64, 3, GVA_MMA_WPG64, false>(cfg, st, sm_count, smem_optin, p, B, max_seq_len,
                                                                     num_splits, max_blocks, stream, n_blocks_out);
        return launch_mma_t<64, 24, 32, 3, GVA_MMA_WPG64, false>(cfg, st, sm_count, smem_optin, p, B, max_seq_len,
                                                                 num_splits, max_blocks, stream, n_blocks_out);
    }
    if (cfg.d_r == 0 && !GQA) {       // value-only cache
        if (cfg.d_v == 64 && *tile_out == 64)
            return launch_mma_t<64, 0, 64, 3, GVA_MMA_WPG64, false>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits,
                                                                    max_blocks, stream, n_blocks_out);
        if (cfg.d_v == 64)
            return launch_mma_t<64, 0, 32, 3, GVA_MMA_WPG64, false>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits,
                                                                    max_blocks, stream, n_blocks_out);
        return launch_mma_t<128, 0, 32, 3, 1, false>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks,
                                                     stream, n_blocks_out);
    }
    if (cfg.d_v == 64 && *tile_out == 64)
        return launch_mma_t<64, 16, 64, 3, GVA_MMA_WPG64, GQA>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks,
                                                   stream, n_blocks_out);
    if (cfg.d_v == 64)
        return launch_mma_t<64, 16, 32, 3, GVA_MMA_WPG64, GQA>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks,
                                                   stream, n_blocks_out);
    return launch_mma_t<128, 32, GQA ? 16 : 32, 3, 1, GQA>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits,
                                                           max_blocks, stream, n_blocks_out);
}

// Multi-token decode (q_len = 2 or 4 new tokens per sequence) on the same kernel: see decode_mma_kernel.
inline int launch_decode_mma_multi(const gva_config &cfg, MmaHostState &st, int sm_count, int smem_optin, const DecodeParams &p,
                                   int B, int q_len, int max_seq_len, int num_splits, int max_blocks, cudaStream_t stream,
                                   int *n_blocks_out, int *tile_out, int *rec_mult_out) {
    if (!mma_supported(cfg, false) || q_len < 2 || q_len > 8) return GVA_ERR_UNSUPPORTED;
    if (q_len > 4) {       // five to eight new tokens: two consumer warps per group share each tile's columns; one block per SM with a deeper ring
        if (!(cfg.d_v == 64 && cfg.G <= 4 && cfg.page_size % 64 == 0)) return GVA_ERR_UNSUPPORTED;
        if ((uint64_t)p.num_pages * cfg.G * cfg.page_size >= (1ull << 31)) return GVA_ERR_UNSUPPORTED;
        *tile_out = 64;
        *rec_mult_out = 1;
        if (cfg.d_r == 24)
            return launch_mma_t<64, 24, 64, 5, 1, false, 4, 2>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, stream, n_blocks_out);
        if (cfg.d_r == 16)
            return launch_mma_t<64, 16, 64, 5, 1, false, 4, 2>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, stream, n_blocks_out);
        if (cfg.d_r == 0)
            return launch_mma_t<64, 0, 64, 5, 1, false, 4, 2>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, stream, n_blocks_out);
        return GVA_ERR_UNSUPPORTED;
    }
    if (!((cfg.d_v == 64 && (cfg.d_r == 16 || cfg.d_r == 24 || cfg.d_r == 0)) || (cfg.d_v == 128 && (cfg.d_r == 32 || cfg.d_r == 0)))) return GVA_ERR_UNSUPPORTED;
    if ((uint64_t)p.num_pages * cfg.G * cfg.page_size >= (1ull << 31)) return GVA_ERR_UNSUPPORTED;
    *tile_out = mma_tile_for(cfg, false);
    if (cfg.d_r == 24) {                // 48-byte positional rows: the 64-token tile only
        if (*tile_out != 64) return GVA_ERR_UNSUPPORTED;
        *rec_mult_out = 1;
        if (q_len == 2)
            return launch_mma_t<64, 24, 64, 3, 1, false, 2>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, stream, n_blocks_out);
        return launch_mma_t<64, 24, 64, 3, 1, false, 4>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, stream, n_blocks_out);
    }
    *rec_mult_out = 1;
#define GVA_MULTI(DV_, DR_, TILE_, QL_)                                                                                       \
    return launch_mma_t<DV_, DR_, TILE_, 3, 1, false, QL_>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, max_blocks, \
                                                            stream, n_blocks_out)
    if (cfg.d_r == 0) {                 // value-only cache
        if (cfg.d_v == 64 && *tile_out == 64) {
            if (q_len == 2) GVA_MULTI(64, 0, 64, 2);
            GVA_MULTI(64, 0, 64, 4);
        }
        if (cfg.d_v == 64) {
            if (q_len == 2) GVA_MULTI(64, 0, 32, 2);
            GVA_MULTI(64, 0, 32, 4);
        }
        if (q_len == 2) GVA_MULTI(128, 0, 32, 2);
        GVA_MULTI(128, 0, 32, 4);
    }
    if (cfg.d_v == 64 && *tile_out == 64) {
        if (q_len == 2) GVA_MULTI(64, 16, 64, 2);
        GVA_MULTI(64, 16, 64, 4);       // three tokens run in the four-token kernel with one slot empty
    }
    if (cfg.d_v == 64) {
        if (q_len == 2) GVA_MULTI(64, 16, 32, 2);
        GVA_MULTI(64, 16, 32, 4);
    }
    if (q_len == 2) GVA_MULTI(128, 32, 32, 2);
    GVA_MULTI(128, 32, 32, 4);
#undef GVA_MULTI
}

}  // namespace gva
