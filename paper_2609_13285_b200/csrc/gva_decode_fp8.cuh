// Split-KV decode over an 8-bit (e4m3) GVA cache: the tensor-core kernel of gva_decode_mma.cuh with the cache tile in
// one byte per element.  Work partition, producer, barriers, partial records and merge are the same; what differs is
// the consumer's way from shared memory to MMA fragments.  The byte MMA (m16n8k32, e4m3 operands) is not a native
// warp-level instruction on this architecture (the compiler widens its operands and splits it: measured slower), so
// the cache bytes are widened to f16 -- exactly: every e4m3 value is an f16 value -- with cvt.rn.f16x2.e4m3x2, two
// codes per instruction, and multiplied with f16 hi/lo halves of the f32 query and weights (m16n8k16, f16 in, f32
// accumulate).  For the score product ldmatrix delivers four consecutive dims of one token per register; for the
// value product the byte-transposing 16x16 ldmatrix delivers four tokens of one dim per register, so both sides
// need nothing but the two conversions per register.  The k index inside an MMA is then a fixed permutation of the
// dims (score product) or tokens (value product); the other operand's fragments are built in the same order.
// Shapes: (d_v, d_r) = (64, 16), (64, 0) with 64-token tiles; (128, 32), (128, 0) with 32-token tiles.
#pragma once

#include "gva_decode_mma.cuh"

// build-time knobs: ring depth, warps per value group (G <= 4), resident blocks per SM the grid is sized for
#ifndef GVA_FP8_NSTAGE
#define GVA_FP8_NSTAGE 3
#endif
#ifndef GVA_FP8_WPG
#define GVA_FP8_WPG 1
#endif
// resident five-warp blocks per SM of the multi-token variants (measured on the long-context workload: 2 tokens
// 79 / 79 / 68 us with 2 / 3 / 4 blocks, 4 tokens 98 / 128 / 142 us: the 4-token variant needs its 168 registers)
#define GVA_FP8_QL_BLOCKS(QL_) ((QL_) == 2 ? 4 : 2)
#ifndef GVA_FP8_BLOCKS_PER_SM
#define GVA_FP8_BLOCKS_PER_SM 4
#endif

namespace gva {

template <int DV_, int DR_, int TILE_>
struct Fp8Traits {
    static constexpr int DV = DV_, DR = DR_, TILE = TILE_;
    static_assert((DV == 64 || DV == 128) && (DR == 0 || DR == 16 || DR == 32) && TILE % 16 == 0, "shape not built");
    static constexpr int VTILE_BYTES = TILE * DV;               // one group's tile: rows of d_v bytes, swizzled over the row width
    static constexpr int KR_ROW = DR;                           // 16 bytes (unswizzled) or 32 bytes (32-byte swizzle)
    static constexpr int KR_BYTES = TILE * KR_ROW;
    static constexpr int KSTEPS_V = DV / 16, KSTEPS = KSTEPS_V + DR / 16;
    static constexpr int MT = DV / 16;
    static constexpr int CHUNKS = TILE / 16;
    static constexpr int DQ = DV + DR;
    // the positional tile is padded to a multiple of 1 KB so that every stage starts on the swizzle period
    __host__ __device__ static constexpr int stage_bytes(int G) { return G * VTILE_BYTES + (KR_BYTES + 1023) / 1024 * 1024; }
    // 16-byte piece c of value row t sits at piece c ^ swz(t): the 64- and 128-byte TMA swizzles
    __host__ __device__ static constexpr uint32_t swz(int t) { return DV == 64 ? ((t >> 1) & 3) : (t & 7); }
    // ... and of positional row t (32-byte rows, 32-byte swizzle; 16-byte rows are one piece)
    __host__ __device__ static constexpr uint32_t swz_kr(int t) { return DR == 32 ? ((t >> 2) & 1) : 0; }
    __host__ __device__ static constexpr int tail_bytes(int B, int nstage) {
        return nstage * 16 /* barriers */ + nstage * 16 /* per-stage meta */ + 16 /* abort */ + (B + 1) * 4;
    }
};

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// four e4m3 codes -> f16 pairs (exact) of the low and of the high half-word
__device__ __forceinline__ void e4m3x4_to_f16x2(uint32_t x, uint32_t &lo, uint32_t &hi) {
    asm("{\n .reg .b16 l, h;\n mov.b32 {l, h}, %2;\n cvt.rn.f16x2.e4m3x2 %0, l;\n cvt.rn.f16x2.e4m3x2 %1, h;\n}\n" : "=r"(lo), "=r"(hi) : "r"(x));
}
// Two 16x16 byte matrices, transposed on the way: lanes 0-15 give the row addresses (16 bytes each) of the first,
// lanes 16-31 of the second.  Lane (g = lane / 4, t = lane % 4) receives bytes [column g | g + 8][rows 4 t .. 4 t + 3]
// of the first matrix in r[0] | r[1] and of the second in r[2] | r[3].
__device__ __forceinline__ void ldsm_b8_x2_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// (x0, x1) -> (hi, lo) f16 pairs of each, two values per conversion instruction
__device__ __forceinline__ void split_pair_hi_lo_f16(float x0, float x1, uint32_t &s0, uint32_t &s1) {
    const __half2 h = __floats2half2_rn(x0, x1);
    const float2 f = __half22float2(h);
    const __half2 l = __floats2half2_rn(x0 - f.x, x1 - f.y);
    const uint32_t hu = *reinterpret_cast<const uint32_t *>(&h), lu = *reinterpret_cast<const uint32_t *>(&l);
    s0 = __byte_perm(hu, lu, 0x5410);
    s1 = __byte_perm(hu, lu, 0x7632);
}
// x = hi + lo with hi, lo f16; hi in the low half-word, lo in the high half-word (|x| must stay below 65504)
__device__ __forceinline__ uint32_t split_hi_lo_f16(float x) {
    const __half hi = __float2half_rn(x);
    const __half lo = __float2half_rn(x - __half2float(hi));
    return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}

// QL > 1 (multi-token decode, QL = 2 or 4 new tokens per sequence): as in the 16-bit kernel, the 4 heads x QL tokens of a
// group are the MMA columns (plain f16 queries and weights, no hi/lo halves), slot s attends to seq_len - (QL - 1 - s)
// tokens, and the partial records and outputs use QL * H pseudo-heads, slot * H + head.
// GQA = true (the matched GQA cache in 8 bits, single token only): a stage holds G key tiles behind the G value tiles and
// no positional tile; the score product reads group g's key tile, the value product its value tile.
template <int DV, int DR, int TILE, int NSTAGE, int WPG, int GMAX, int QL = 1, bool GQA = false>
__global__ void __launch_bounds__(32 * (GMAX * WPG + 1), GMAX <= 4 ? (QL == 1 ? GVA_FP8_BLOCKS_PER_SM : GVA_FP8_QL_BLOCKS(QL)) : (QL == 1 ? 2 : 1))      // register caps: 4 five-warp blocks (d_v = 64) or 2 nine-warp blocks (d_v = 128) per SM
decode_fp8_kernel(DecodeParams p, const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_k) {
    using T = Fp8Traits<DV, DR, TILE>;
    constexpr int CPW = T::CHUNKS / WPG;          // 16-token chunks per consumer warp and tile
    static_assert(CPW >= 1 && CPW * WPG == T::CHUNKS, "tile must split evenly over the group's warps");
    grid_dependency_launch();
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // dynamic shared memory is only guaranteed 16-byte aligned: round up to the swizzle atom
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int G = p.G, H = p.H;
    static_assert(QL == 1 || QL == 2 || QL == 4, "multi-token decode: 2 or 4 new tokens");
    static_assert(!GQA || (QL == 1 && DR == 0), "the GQA cache: single-token decode, no positional slice");
    constexpr int NBK = QL == 1 ? 1 : QL / 2;     // N-blocks of 8 columns
    const int ql = QL == 1 ? 1 : p.q_len;         // new tokens per sequence actually present (<= QL; the other slots stay empty)
    const int HQ = H * ql;                        // pseudo-heads of the partial records
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n_consumers = G * WPG;
    const int stage_bytes = GQA ? 2 * G * T::VTILE_BYTES : T::stage_bytes(G);

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
    // Early start: as in the 16-bit kernel (see decode_mma_kernel).
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
        // nothing to stream: an empty split still owns its records (weight 0 in the merge)
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
                        if constexpr (GQA) tma_load_2d_stream(base + (G + g) * T::VTILE_BYTES, &tm_k, 0, (int)((page * G + g) * p.P + slot0), bar, pol);
                        tma_load_2d_stream(base + g * T::VTILE_BYTES, &tm_v, 0, (int)((page * G + g) * p.P + slot0), bar, pol);
                    }
                });
        }
    } else {
        // ============ consumer: value group g, token chunks [part*CPW, part*CPW + CPW) of every tile ============
        const int g = warp / WPG;
        const int part = warp % WPG;
        const int jh = lane & 3;          // head within the group this lane's score/output columns belong to
        const int r8 = lane >> 2;         // row within an 8-row block
        // Fragment addressing inside a 16-token chunk of the value tile (64-byte rows, 64-byte swizzle: 16-byte piece c
        // of row t sits at piece c ^ ((t >> 1) & 3)).  The token order inside a chunk is free on both products as long as
        // they agree; it is chosen so that every 8 rows fetched together differ in t mod 8 (no bank conflicts).  With
        // pi(j) = j (j < 8), j ^ 2 (j >= 8):
        //   value product: the transposing load's row j is token pi(j); a register holds tokens pi(4t .. 4t + 3) of one dim,
        //                  its low half becomes k = 2t, 2t + 1 and its high half k = 2t + 8, 2t + 9 of the MMA
        //   score product: MMA row g is token pi(4 (g / 2) + g % 2), row g + 8 is token pi(4 (g / 2) + 2 + g % 2), so that the
        //                  weights of rows (2t, 2t + 1), which the register transpose brings together, are k = 2t, 2t + 1
        //                  (from the low rows) and k = 2t + 8, 2t + 9 (from the high rows)
        const int r7 = lane & 7;
        auto pi = [](int j) { return j < 8 ? j : (j ^ 2); };
        const int row_qk = pi(4 * (r7 >> 1) + 2 * ((lane >> 3) & 1) + (r7 & 1));    // x4: (low | high rows) x (piece 2i | 2i + 1)
        const int ch_ld = lane >> 4;
        const uint32_t off_qk = row_qk * DV, swz_qk = T::swz(row_qk);
        const uint32_t off_kr = row_qk * T::KR_ROW, swz_kr = T::swz_kr(row_qk);
        const int row_pv = pi(lane & 15);                                            // x2: (piece 2i | 2i + 1), 16 tokens each
        const uint32_t off_pv = row_pv * DV, swz_pv = T::swz(row_pv);
        const int tok_lo = pi(4 * (r8 >> 1) + (r8 & 1)), tok_hi = pi(4 * (r8 >> 1) + 2 + (r8 & 1));   // this lane's two score rows
        if constexpr (QL == 1) {
        uint32_t qf[T::KSTEPS][2];        // B fragments of Q^T as f16: column n = lane/4 = 2*head + {hi, lo}; k-step kk covers
                                          // dims 16 kk .. 16 kk + 15 in the order the converted A registers present them
        float oacc[T::MT][4];
        float m_run = -INFINITY, l_run = 0.f;
        const float scale = p.scale_log2;
        const int lo_part = r8 & 1;

        // absorbed query of head (lane/4)/2, hi or lo part by (lane/4)&1, as mma B fragments: b0 = dims 4 jh, 4 jh + 1 and
        // b1 = dims 4 jh + 2, 4 jh + 3 of the k-step's 16 dims (the A registers carry the cache bytes in that order)
        auto load_query = [&](int b) {
            const float *q = p.q + ((size_t)b * H + g * kHeadsPerGroup + (r8 >> 1)) * T::DQ;
#pragma unroll
            for (int kk = 0; kk < T::KSTEPS; ++kk) {
                const float4 v = *reinterpret_cast<const float4 *>(q + kk * 16 + 4 * jh);
                const uint32_t sx = split_hi_lo_f16(v.x), sy = split_hi_lo_f16(v.y), sz = split_hi_lo_f16(v.z), sw = split_hi_lo_f16(v.w);
                qf[kk][0] = lo_part ? ((sx >> 16) | (sy & 0xffff0000u)) : ((sx & 0xffffu) | (sy << 16));
                qf[kk][1] = lo_part ? ((sz >> 16) | (sw & 0xffff0000u)) : ((sz & 0xffffu) | (sw << 16));
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
                // rows past the sequence end may hold anything (the NaN code included): zero this warp's share of them
                // so that a zero weight times such a row stays zero
                const int z0 = max(n_valid, row0);
                const int n_zero_chunks = (row0 + CPW * 16 - z0) * (DV / 16);
                for (int c = lane; c < n_zero_chunks; c += 32)
                    *reinterpret_cast<uint4 *>(vt + (z0 + c / (DV / 16)) * DV + (c % (DV / 16)) * 16) = make_uint4(0, 0, 0, 0);
                // generic-proxy writes must be ordered before the TMA write that later refills the stage
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                __syncwarp();
            }
            const uint32_t vt_u32 = smem_u32(vt) + row0 * DV;
            const uint32_t ks_u32 = GQA ? smem_u32(stage + (size_t)(G + g) * T::VTILE_BYTES) + row0 * DV : vt_u32;   // score source
            uint32_t a_qk[DV / 32], a_pv[DV / 32];            // per pair of pieces: this lane's row address within a chunk
#pragma unroll
            for (int pr = 0; pr < DV / 32; ++pr) {
                a_qk[pr] = ks_u32 + off_qk + ((((uint32_t)(2 * pr + ch_ld)) ^ swz_qk) << 4);
                a_pv[pr] = vt_u32 + off_pv + ((((uint32_t)(2 * pr + ch_ld)) ^ swz_pv) << 4);
            }
            const uint32_t kr_u32 = smem_u32(stage + (size_t)G * T::VTILE_BYTES) + row0 * T::KR_ROW;

            // ---- S^T = V_tile . Q^T (+ positional part), 16 tokens per m-tile ----
            float sacc[CPW][4];
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sacc[c][e] = 0.f;
#pragma unroll
                for (int pr = 0; pr < DV / 32; ++pr) {        // two 16-dim chunks per fetch
                    uint32_t r[4];                             // (tok r8, chunk 2 pr) (tok r8 + 8, chunk 2 pr) (tok r8, chunk 2 pr + 1) (tok r8 + 8, ..)
                    ldsm_x4(a_qk[pr] + c * 16 * DV, r);
#pragma unroll
                    for (int hx = 0; hx < 2; ++hx) {
                        uint32_t a[4];
                        e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                        e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
                        mma_f16(sacc[c], a, qf[2 * pr + hx][0], qf[2 * pr + hx][1]);
                    }
                }
                if constexpr (DR == 16) {   // the positional key: 16-byte rows, one fetch of (low | high rows)
                    uint32_t r[2];
                    ldsm_x2(kr_u32 + c * 16 * T::KR_ROW + off_kr, r);        // lanes 0-7: low rows, 8-15: high rows
                    uint32_t a[4];
                    e4m3x4_to_f16x2(r[0], a[0], a[2]);
                    e4m3x4_to_f16x2(r[1], a[1], a[3]);
                    mma_f16(sacc[c], a, qf[T::KSTEPS_V][0], qf[T::KSTEPS_V][1]);
                } else if constexpr (DR == 32) {   // 32-byte rows: (low | high rows) x (piece 0 | 1)
                    uint32_t r[4];
                    ldsm_x4(kr_u32 + c * 16 * T::KR_ROW + off_kr + ((((uint32_t)ch_ld) ^ swz_kr) << 4), r);
#pragma unroll
                    for (int hx = 0; hx < 2; ++hx) {
                        uint32_t a[4];
                        e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                        e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
                        mma_f16(sacc[c], a, qf[T::KSTEPS_V + hx][0], qf[T::KSTEPS_V + hx][1]);
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
                    if (row0 + c * 16 + tok_lo >= n_valid) sr[c][0] = -INFINITY;
                    if (row0 + c * 16 + tok_hi >= n_valid) sr[c][1] = -INFINITY;
                }
                tmax = fmaxf(tmax, fmaxf(sr[c][0], sr[c][1]));
            }
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 8));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
            const float m_new = fmaxf(m_run, tmax * scale);          // scale > 0: max commutes with it
            const bool live = m_new != -INFINITY;
            const float m_use = live ? m_new : 0.f;                  // keeps (-inf) - (-inf) out of the exponent
            if (__any_sync(0xffffffffu, m_new != m_run)) {           // rare once the running maxima have settled
                const float corr = fast_exp2(m_run - m_use);         // 2^(-inf) = 0 for the first live tile
                l_run *= corr;
#pragma unroll
                for (int mt = 0; mt < T::MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) oacc[mt][e] *= corr;
            }
            m_run = m_new;

            // ---- O^T += V_tile^T . P^T: m-tile mt holds value dims 16 mt .. 16 mt + 15 ----
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                const float p0 = fast_exp2(fmaf(sr[c][0], scale, -m_use));
                const float p1 = fast_exp2(fmaf(sr[c][1], scale, -m_use));
                l_run += p0 + p1;
                // (hi, lo) of p for this lane's two token rows and columns 2*jh, 2*jh+1 -> transpose to B fragments
                uint32_t s0, s1;
                split_pair_hi_lo_f16(p0, p1, s0, s1);
                const uint32_t pb0 = movmatrix_trans(s0);
                const uint32_t pb1 = movmatrix_trans(s1);
#pragma unroll
                for (int pr = 0; pr < DV / 32; ++pr) {
                    uint32_t r[4];    // dims 32 pr + (r8 | r8 + 8) and 32 pr + 16 + (r8 | r8 + 8), tokens pi(4 jh .. 4 jh + 3) each
                    ldsm_b8_x2_trans(a_pv[pr] + c * 16 * DV, r);
#pragma unroll
                    for (int hx = 0; hx < 2; ++hx) {
                        uint32_t a[4];
                        e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                        e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
                        mma_f16(oacc[2 * pr + hx], a, pb0, pb1);
                    }
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
                for (int mt = 0; mt < T::MT; ++mt)
                {
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
            uint32_t qf[T::KSTEPS][NBK][2];   // B fragments of Q^T (f16): column n = lane / 4 of N-block nb, dims in the
                                              // order the converted A registers present them
            uint32_t qlo[T::KSTEPS][NBK][2];  // ... and of q - f16(q): the score product is taken with both, so that a score of
                                              // any size is as exact as the cache's codes allow (with the first half alone a
                                              // score s is off by about |s| 2^-12, which breaks the contract on peaked rows)
            float oacc[T::MT][NBK][4];
            float m_run[NBK][2], l_run[NBK][2];   // per column of this lane: columns 2 jh, 2 jh + 1 of every N-block
            const float scale = p.scale_log2;
            // the lane's B-fragment column n = lane / 4 = r8 is (slot 2 nb + n / 4, head n % 4)
            int cur_ql = ql;                       // new tokens of the current sequence
            auto load_query = [&](int b) {
                size_t row0q = (size_t)b * ql;
                cur_ql = ql;
                if (p.cu_q) {                      // its own count and first query row per sequence
                    const int r_lo = p.cu_q[b];
                    row0q = (size_t)r_lo;
                    cur_ql = min(max(p.cu_q[b + 1] - r_lo, 0), ql);
                }
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb) {
                    const int slot = 2 * nb + (r8 >> 2), head = r8 & 3;
                    const bool present = slot < cur_ql;   // an absent slot gets a zero query; its columns are masked everywhere
                    const float *q = p.q + ((row0q + (present ? slot : 0)) * H + g * kHeadsPerGroup + head) * T::DQ;
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS; ++kk) {
                        float4 v = *reinterpret_cast<const float4 *>(q + kk * 16 + 4 * jh);
                        if (!present) v = make_float4(0.f, 0.f, 0.f, 0.f);
                        const __half2 w0 = __floats2half2_rn(v.x, v.y), w1 = __floats2half2_rn(v.z, v.w);
                        const float2 f0 = __half22float2(w0), f1 = __half22float2(w1);
                        const __half2 l0 = __floats2half2_rn(v.x - f0.x, v.y - f0.y), l1 = __floats2half2_rn(v.z - f1.x, v.w - f1.y);
                        qf[kk][nb][0] = *reinterpret_cast<const uint32_t *>(&w0);
                        qf[kk][nb][1] = *reinterpret_cast<const uint32_t *>(&w1);
                        qlo[kk][nb][0] = *reinterpret_cast<const uint32_t *>(&l0);
                        qlo[kk][nb][1] = *reinterpret_cast<const uint32_t *>(&l1);
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
                    const int n_zero_chunks = (row0 + CPW * 16 - z0) * (DV / 16);
                    for (int c = lane; c < n_zero_chunks; c += 32)
                        *reinterpret_cast<uint4 *>(vt + (z0 + c / (DV / 16)) * DV + (c % (DV / 16)) * 16) = make_uint4(0, 0, 0, 0);
                    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    __syncwarp();
                }
                const bool masked = reach < row0 + CPW * 16 || cur_ql < QL;  // some slot does not see the whole share of this warp
                const uint32_t vt_u32 = smem_u32(vt) + row0 * DV;
                const uint32_t kr_u32 = smem_u32(stage + (size_t)G * T::VTILE_BYTES) + row0 * T::KR_ROW;
                uint32_t a_qk[DV / 32], a_pv[DV / 32];
#pragma unroll
                for (int pr = 0; pr < DV / 32; ++pr) {
                    a_qk[pr] = vt_u32 + off_qk + ((((uint32_t)(2 * pr + ch_ld)) ^ swz_qk) << 4);
                    a_pv[pr] = vt_u32 + off_pv + ((((uint32_t)(2 * pr + ch_ld)) ^ swz_pv) << 4);
                }

                // ---- S^T = V_tile . Q^T (+ positional part): 16 tokens per m-tile, 8 columns per N-block ----
                float sacc[CPW][NBK][4];
#pragma unroll
                for (int c = 0; c < CPW; ++c) {
#pragma unroll
                    for (int nb = 0; nb < NBK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) sacc[c][nb][e] = 0.f;
#pragma unroll
                    for (int pr = 0; pr < DV / 32; ++pr) {
                        uint32_t r[4];
                        ldsm_x4(a_qk[pr] + c * 16 * DV, r);
#pragma unroll
                        for (int hx = 0; hx < 2; ++hx) {
                            uint32_t a[4];
                            e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                            e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
#pragma unroll
                            for (int nb = 0; nb < NBK; ++nb) {
                                mma_f16(sacc[c][nb], a, qlo[2 * pr + hx][nb][0], qlo[2 * pr + hx][nb][1]);
                                mma_f16(sacc[c][nb], a, qf[2 * pr + hx][nb][0], qf[2 * pr + hx][nb][1]);
                            }
                        }
                    }
                    if constexpr (DR == 16) {
                        uint32_t r[2];
                        ldsm_x2(kr_u32 + c * 16 * T::KR_ROW + off_kr, r);
                        uint32_t a[4];
                        e4m3x4_to_f16x2(r[0], a[0], a[2]);
                        e4m3x4_to_f16x2(r[1], a[1], a[3]);
#pragma unroll
                        for (int nb = 0; nb < NBK; ++nb) {
                            mma_f16(sacc[c][nb], a, qlo[T::KSTEPS_V][nb][0], qlo[T::KSTEPS_V][nb][1]);
                            mma_f16(sacc[c][nb], a, qf[T::KSTEPS_V][nb][0], qf[T::KSTEPS_V][nb][1]);
                        }
                    } else if constexpr (DR == 32) {
                        uint32_t r[4];
                        ldsm_x4(kr_u32 + c * 16 * T::KR_ROW + off_kr + ((((uint32_t)ch_ld) ^ swz_kr) << 4), r);
#pragma unroll
                        for (int hx = 0; hx < 2; ++hx) {
                            uint32_t a[4];
                            e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                            e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
#pragma unroll
                            for (int nb = 0; nb < NBK; ++nb) {
                                mma_f16(sacc[c][nb], a, qlo[T::KSTEPS_V + hx][nb][0], qlo[T::KSTEPS_V + hx][nb][1]);
                                mma_f16(sacc[c][nb], a, qf[T::KSTEPS_V + hx][nb][0], qf[T::KSTEPS_V + hx][nb][1]);
                            }
                        }
                    }
                }
                // ---- online softmax per column: this lane holds columns 2 jh, 2 jh + 1 of every N-block at its two token
                //      rows of every m-tile; both columns belong to slot 2 nb + jh / 2 ----
                float corr[NBK][2], m_use[NBK][2];
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb) {
                    const int slot_l = 2 * nb + (jh >> 1);
                    const int lim = slot_l < cur_ql ? reach + slot_l : 0;     // tokens of the tile this slot sees (an absent slot: none)
                    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < CPW; ++c) {
                        if (masked) {
                            if (row0 + c * 16 + tok_lo >= lim) sacc[c][nb][0] = sacc[c][nb][1] = -INFINITY;
                            if (row0 + c * 16 + tok_hi >= lim) sacc[c][nb][2] = sacc[c][nb][3] = -INFINITY;
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
                        const float p00 = fast_exp2(fmaf(sacc[c][nb][0], scale, -m_use[nb][0]));   // low row,  column 2 jh
                        const float p01 = fast_exp2(fmaf(sacc[c][nb][1], scale, -m_use[nb][1]));   // low row,  column 2 jh + 1
                        const float p10 = fast_exp2(fmaf(sacc[c][nb][2], scale, -m_use[nb][0]));   // high row, column 2 jh
                        const float p11 = fast_exp2(fmaf(sacc[c][nb][3], scale, -m_use[nb][1]));
                        l_run[nb][0] += p00 + p10;
                        l_run[nb][1] += p01 + p11;
                        const __half2 w0 = __floats2half2_rn(p00, p01), w1 = __floats2half2_rn(p10, p11);
                        pb[nb][0] = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&w0));
                        pb[nb][1] = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&w1));
                    }
#pragma unroll
                    for (int pr = 0; pr < DV / 32; ++pr) {
                        uint32_t r[4];
                        ldsm_b8_x2_trans(a_pv[pr] + c * 16 * DV, r);
#pragma unroll
                        for (int hx = 0; hx < 2; ++hx) {
                            uint32_t a[4];
                            e4m3x4_to_f16x2(r[2 * hx], a[0], a[2]);
                            e4m3x4_to_f16x2(r[2 * hx + 1], a[1], a[3]);
#pragma unroll
                            for (int nb = 0; nb < NBK; ++nb) mma_f16(oacc[2 * pr + hx][nb], a, pb[nb][0], pb[nb][1]);
                        }
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
                            const int col = 2 * jh + e;                       // column of N-block nb: slot 2 nb + col / 4, head col % 4
                            if (2 * nb + (col >> 2) >= cur_ql) continue;       // (uniform over the lanes that reduce together)
                            const size_t rh = (size_t)rec * HQ + (size_t)(2 * nb + (col >> 2)) * H + g * kHeadsPerGroup + (col & 3);
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


// ---- host ---------------------------------------------------------------------------------------------
inline bool fp8_supported(const gva_config &cfg) {
    const bool shape = (cfg.d_v == 64 && (cfg.d_r == 16 || cfg.d_r == 0)) || (cfg.d_v == 128 && (cfg.d_r == 32 || cfg.d_r == 0));
    return cfg.cache_dtype == GVA_E4M3 && shape && cfg.page_size % 64 == 0 && cfg.G <= 8;
}
// resident blocks per SM the grid (and the workspace) is sized for: as many as measured best where the rings fit
inline int fp8_blocks_per_sm(const gva_config &cfg) { return (cfg.d_v == 128 && cfg.G > 4) ? 2 : GVA_FP8_BLOCKS_PER_SM; }
inline int fp8_tile(const gva_config &cfg) { return cfg.d_v == 64 ? 64 : 32; }

inline bool encode_map_u8(const MmaHostState &st, CUtensorMap *map, const void *base, uint64_t inner, uint64_t rows,
                          uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz) {
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return st.encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DV, int DR, int TILE, int QL = 1, bool GQA = false>
int launch_fp8_t(const gva_config &cfg, MmaHostState &st, int sm_count, int smem_optin, const DecodeParams &p, int B,
                 int max_seq_len, int num_splits, cudaStream_t stream, int *n_blocks_out) {
    using T = Fp8Traits<DV, DR, TILE>;
    constexpr int NSTAGE = GVA_FP8_NSTAGE;
    constexpr int wpg = GVA_FP8_WPG;      // warps per group (each takes 1 / wpg of a tile's tokens); one measured fastest
    const int G = cfg.G;
    if (G * wpg + 1 > 9) return GVA_ERR_UNSUPPORTED;
    const size_t stage = GQA ? (size_t)2 * G * T::VTILE_BYTES : (size_t)T::stage_bytes(G);
    const size_t smem = 1024 + (size_t)NSTAGE * stage + T::tail_bytes(B, NSTAGE) + 16;
    if (smem > (size_t)smem_optin) return GVA_ERR_UNSUPPORTED;
    auto fn = G <= 4 ? decode_fp8_kernel<DV, DR, TILE, NSTAGE, wpg, 4, QL, GQA> : decode_fp8_kernel<DV, DR, TILE, NSTAGE, wpg, 8, QL, GQA>;
    static int s_smem_set[2][kMaxDevicesCached] = {};      // per (G <= 4 or not, device): the attribute is set once, not per call
    const int dev = st.device >= 0 && st.device < kMaxDevicesCached ? st.device : 0;
    if (s_smem_set[G <= 4][dev] != (int)smem || st.device >= kMaxDevicesCached) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GVA_ERR_CUDA;
        s_smem_set[G <= 4][dev] = (int)smem;
    }
    const void *second = GQA ? p.k_pool : p.kr_pool;
    const MapPair *mp = st.find(p.v_pool, second, p.num_pages, GQA ? 3 : 2);
    if (!mp) {
        MapPair *m = st.slot_for(p.v_pool, second, p.num_pages, GQA ? 3 : 2);
        bool ok = encode_map_u8(st, &m->tm_v, p.v_pool, DV, (uint64_t)p.num_pages * G * p.P, DV, TILE,
                                DV == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B);
        if (ok && GQA) ok = encode_map_u8(st, &m->tm_k, p.k_pool, DV, (uint64_t)p.num_pages * G * p.P, DV, TILE,
                                          DV == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B);
        else if (ok && DR == 0) m->tm_k = m->tm_v;      // value-only cache: no positional tile (the kernel never uses this map)
        else if (ok) ok = encode_map_u8(st, &m->tm_k, p.kr_pool, DR, (uint64_t)p.num_pages * p.P, DR, TILE,
                                        DR == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE);
        if (!ok) {
            st.forget_last();
            return GVA_ERR_CUDA;
        }
        mp = m;
    }
    const int threads = 32 * (G * wpg + 1);
    int grid;
    if (num_splits > 0) {
        grid = B * num_splits;
    } else {
        const long long tiles_ub = (long long)B * ((max_seq_len + TILE - 1) / TILE);
        // what the workspace is sized for; the multi-token variants: four (2 tokens) or two (4 tokens) five-warp blocks,
        // or one nine-warp block per SM
        const int per_sm = GQA ? (DV == 64 && G <= 4 ? 2 : 1)      // twice the tiles per stage: what the shared memory of an SM holds
                               : QL == 1 ? fp8_blocks_per_sm(cfg) : (G > 4 ? 1 : GVA_FP8_QL_BLOCKS(QL));
        const long long want = (long long)per_sm * sm_count;
        grid = (int)(tiles_ub < want ? (tiles_ub < 1 ? 1 : tiles_ub) : want);
    }
    *n_blocks_out = grid;
    if (st.dry) return GVA_OK;
    DecodeParams pp = p;
    pp.rec_mult = wpg;
    if (launch_pdl(fn, dim3(grid), dim3(threads), smem, stream, pp, mp->tm_v, mp->tm_k) != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

inline int launch_decode_fp8(const gva_config &cfg, MmaHostState &st, int sm_count, int smem_optin, const DecodeParams &p, int B,
                             int q_len, int max_seq_len, int num_splits, cudaStream_t stream, int *n_blocks_out, int *tile_out,
                             int *rec_mult_out, bool gqa = false) {
    if (!fp8_supported(cfg)) return GVA_ERR_UNSUPPORTED;
    if ((uint64_t)p.num_pages * cfg.G * cfg.page_size >= (1ull << 31)) return GVA_ERR_UNSUPPORTED;
    *tile_out = fp8_tile(cfg);
    *rec_mult_out = GVA_FP8_WPG;
    if (gqa) {             // the matched GQA cache: keys and values of width d_h = d_v per group, single token
        if (q_len > 1) return GVA_ERR_UNSUPPORTED;
        if (cfg.d_v == 64) return launch_fp8_t<64, 0, 64, 1, true>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out);
        return launch_fp8_t<128, 0, 32, 1, true>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out);
    }
    if (q_len > 1) {       // multi-token decode: 2..4 new tokens per sequence, caches with a positional slice
        if (q_len > 4 || cfg.d_r == 0) return GVA_ERR_UNSUPPORTED;
#define GVA_FP8_MULTI(DV_, DR_, TILE_, QL_) \
    return launch_fp8_t<DV_, DR_, TILE_, QL_>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out)
        if (cfg.d_v == 64) {
            if (q_len == 2) GVA_FP8_MULTI(64, 16, 64, 2);
            GVA_FP8_MULTI(64, 16, 64, 4);
        }
        if (q_len == 2) GVA_FP8_MULTI(128, 32, 32, 2);
        GVA_FP8_MULTI(128, 32, 32, 4);
#undef GVA_FP8_MULTI
    }
    if (cfg.d_v == 64)
        return cfg.d_r == 16 ? launch_fp8_t<64, 16, 64>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out)
                             : launch_fp8_t<64, 0, 64>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out);
    return cfg.d_r == 32 ? launch_fp8_t<128, 32, 32>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out)
                         : launch_fp8_t<128, 0, 32>(cfg, st, sm_count, smem_optin, p, B, max_seq_len, num_splits, stream, n_blocks_out);
}

}  // namespace gva
