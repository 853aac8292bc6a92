// Causal prefill / chunked-prefill attention over the paged bf16 GVA cache on the 5th-generation tensor
// cores (tcgen05 + tensor memory), sm_100a.
//
// What it computes (the paper's multi-token form: ordinary causal attention with content + positional scores,
// Section 3.3 and the remark after Algorithm 1), in the absorbed form of Eq. absorb: for query token i at
// position t, head h of group g,
//     s_ij = q~_i,h . v_j,g + q^rope_i,h . k^rope_j   (j <= t),   o_i,h = softmax_j(s_ij / sqrt(d_qk)) V_g.
// With the query absorbed the key of token j is [v_j,g | k^rope_j]: the cached value tile IS the content-key
// tile, so one shared-memory tile feeds both the score product (as a K-major operand) and the value product
// (as an MN-major operand), and the H/G = 4 heads of a group stack into the M dimension of one tile.
//
// Layout of the work
//   thread block   = 32 query tokens x 4 heads of one (sequence, value group): 128 rows = one M = 128 MMA tile
//   warps 0-3      = softmax: thread r owns row r (token r / 4, head r % 4) = tensor-memory lane r
//   warp 4         = one lane: TMA loads of the 64-token value tile and positional-key tile into a ring, and issuer of
//                    the value products
//   warp 5         = one lane: issuer of the score products; the warp owns the tensor-memory allocation
//   per 64-token tile j:
//     S[j & 1]  = Q K_j^T            tcgen05.mma, K = d_v (value dims, 128-byte swizzle) + d_r (RoPE dims)
//     softmax   : tcgen05.ld row -> mask -> row maximum / sum (base 2) -> P_j as bf16 pairs, written over the first
//                 half of the row's own S columns (a row has one reader, so nothing else can still need them)
//     O        += P_j V_j            tcgen05.mma, A = P from tensor memory, B = the same value tile as an MN-major operand
//     O accumulates in tensor memory across tiles.  The softmax reference of a row moves only when the running
//     maximum grows by more than 2^8; only then is that row of O rescaled (read, multiplied, written back).
//   S has two buffers, so the score product of tile j + 1 runs while the softmax warps work on tile j; for d_v = 64
//   the query tile lives in tensor memory too, so every MMA reads only its B operand (the cache tile) from shared
//   memory; two blocks share an SM (256 tensor-memory columns each).  Shared memory carries only operands the tensor
//   core reads (the cache tiles, and Q for d_v = 128): P never touches it.
//   Split-KV (gva_decode_multi: few new tokens over a long context): a query block is shared by several thread
//   blocks, each over a contiguous range of tiles, which leave unnormalised (O, reference, sum) per row for
//   merge_splits_kernel.
//   Rules this file keeps: (1) tcgen05.ld / tcgen05.st are warp-wide (.sync.aligned): they never sit inside a per-lane
//   branch, and every wait that guards them returns a warp-uniform result; (2) every barrier that is waited on by
//   parity is argued, at its wait, never to be two phases ahead of that waiter; (3) every wait is bounded: on expiry
//   the block records GVA_ERR_TIMEOUT, drains what it issued, frees its tensor memory and exits.
#pragma once

#include "gva_decode_mma.cuh"
#include "gva_decode_fp8.cuh"

namespace gva {

struct PrefillParams {
    const float *q_abs;          // [n_q][H][d_v + d_r] absorbed content query, rotated positional query
    const int32_t *cu_q;         // [B + 1] first query row of every sequence
    const int32_t *ctx_lens;     // [B] tokens cached before the chunk
    const int32_t *block_table;  // nullable
    float *out;                  // [n_q][H][d_v]
    float *lse;                  // [n_q][H], nullable
    int32_t *dev_status;         // nullable
    int B, H, G, P, num_pages, max_pages;
    float scale_log2;            // softmax scale * log2(e)
    // split-KV (multi-token decode over a long cached context): every query block is handled by num_splits thread
    // blocks, each over a contiguous range of tiles, which leave unnormalised partial results for merge_splits_kernel
    int num_splits;              // 1 = no split: the kernel writes out / lse itself
    float *part_o;               // [n_q][H][num_splits][d_v]   partial O relative to part_ml[..][0]
    float *part_ml;              // [n_q][H][num_splits][2]     reference (log2 domain) and sum; (-inf, 0) for an empty range
};

// C8 = true: the 8-bit (e4m3) cache.  TMA lands the byte tiles in a raw region of the stage, the producer warp widens them
// to f16 (exact: every e4m3 value is an f16 value) into the same swizzled operand tiles the 16-bit cache is loaded into, and
// every MMA operand of the kernel is f16 instead of bf16 (queries as hi + lo f16, weights as f16).
template <int DV, int DR, bool C8 = false>
struct PrefillTraits {
    static constexpr int QTOK = 32;                              // query tokens per block
    static constexpr int ROWS = QTOK * kHeadsPerGroup;           // 128 = MMA M
    static constexpr int TILE = 64;                              // cached tokens per tile = MMA N of the score product
    static constexpr int NSTAGE = C8 ? 5 : 4;                    // (8-bit cache: one more, so that the tile widened at the top of
                                                                 //  iteration t was requested two iterations earlier)
    static constexpr int BOXES = DV / 64;                        // 64-dim (128-byte) boxes per value row
    static constexpr int QBOX_BYTES = ROWS * 128;
    static constexpr int QV_BYTES = BOXES * QBOX_BYTES;
    static constexpr int DRP = (DR + 15) / 16 * 16;              // RoPE dims as the MMA sees them: d_r = 24 occupies 32, the
                                                                 // last 8 zero (the TMA box is wider than the row and reads
                                                                 // the fill value there; the query's columns are stored as 0)
    static constexpr int KR_ROW = DRP * 2;                       // 32 or 64 bytes
    static constexpr int QR_BYTES = (ROWS * KR_ROW + 1023) & ~1023;
    static constexpr int VBOX_BYTES = TILE * 128;
    static constexpr int V_BYTES = BOXES * VBOX_BYTES;
    static constexpr int KR_BYTES = TILE * KR_ROW;
    static constexpr int KR_PAD = (KR_BYTES + 1023) & ~1023;
    static constexpr int RAW_V_BYTES = C8 ? TILE * DV : 0;        // the byte tiles as TMA delivers them (rows of d_v / d_r bytes, unswizzled)
    static constexpr int RAW_K_BYTES = C8 ? TILE * DR : 0;
    static constexpr int OFF_RAW = V_BYTES + KR_PAD;              // within a stage
    static constexpr int STAGE_BYTES = OFF_RAW + ((RAW_V_BYTES + RAW_K_BYTES + 1023) & ~1023);
    // Tensor-memory columns: two score buffers (64 each; P overwrites the first 32 of its S), O (DV), and the query as bf16
    // pairs -- q = hi + lo, (DV + DR) / 2 columns each: an MMA whose A operand comes from tensor memory reads only B
    // from shared memory (measured: 128 x 64 x 16 MMAs with both operands in shared memory run at 62 cycles each -- the
    // 6 KB of operands per MMA at ~97 B/clk -- against 32 with A in tensor memory).  d_v = 64: two blocks per SM with 256
    // columns each hold hi; lo (40 more columns) does not fit and sits in shared memory.  d_v = 128: the stages alone
    // allow one block per SM, which then takes all 512 columns and holds hi and lo.
    static constexpr int TMEM_COLS = DV == 64 ? 256 : 512;
    static constexpr int NSBUF = 2;
    static constexpr int COL_S = 0, COL_O = NSBUF * TILE, COL_Q = COL_O + DV, COL_QLO = COL_Q + (DV + DRP) / 2;
    static constexpr bool Q_IN_TMEM = COL_Q + (DV + DRP) / 2 <= TMEM_COLS;
    static constexpr bool LO_IN_TMEM = Q_IN_TMEM && COL_QLO + (DV + DRP) / 2 <= TMEM_COLS;
    // Shared memory: whichever of hi (OFF_QV / OFF_QR) and lo (OFF_LOV / OFF_LOR) is not in tensor memory.
    static constexpr int OFF_QV = 0;
    static constexpr int OFF_QR = OFF_QV + (Q_IN_TMEM ? 0 : QV_BYTES);
    static constexpr int OFF_LOV = OFF_QR + (Q_IN_TMEM ? 0 : QR_BYTES);
    static constexpr int OFF_LOR = OFF_LOV + (LO_IN_TMEM ? 0 : QV_BYTES);
    static constexpr int OFF_STAGE = OFF_LOR + (LO_IN_TMEM ? 0 : QR_BYTES);
    static constexpr int OFF_BAR = OFF_STAGE + NSTAGE * STAGE_BYTES;
    static constexpr int N_BARS = 2 * NSTAGE + 9 + (C8 ? NSTAGE : 0);
    static constexpr int SMEM_BYTES = 1024 + OFF_BAR + N_BARS * 8 + 16;
    static_assert(NSBUF * TILE + DV <= TMEM_COLS, "the score buffers and O must fit the allocation");
    static constexpr int BLOCKS_PER_SM = 512 / TMEM_COLS;
    static constexpr int KSTEPS_V = DV / 16, KSTEPS_R = DRP / 16;
    static constexpr int THREADS = 192;
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, f32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same with A read from tensor memory (rows = lanes, two bf16 per 32-bit column, K-major).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
        "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_st16_nowait(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
        "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st32u_nowait(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
        "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]),
        "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]),
        "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st8_nowait(uint32_t taddr, const uint32_t (&v)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n" ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st4_nowait(uint32_t taddr, const uint32_t (&v)[4]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr),
        "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), "f"(v[9]), "f"(v[10]),
        "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]), "f"(v[18]), "f"(v[19]), "f"(v[20]),
        "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]), "f"(v[28]), "f"(v[29]), "f"(v[30]),
        "f"(v[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// 32 consecutive f32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, float (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]), "=f"(v[9]),
          "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]), "=f"(v[17]), "=f"(v[18]),
          "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]), "=f"(v[25]), "=f"(v[26]), "=f"(v[27]),
          "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units), descriptor
// version 1 (bit 46), swizzle mode in bits 61-63 (2 = 128-byte, 4 = 64-byte, 6 = 32-byte).
constexpr uint64_t kSwz128 = 2, kSwz64 = 4, kSwz32 = 6;
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t swizzle) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (swizzle << 61);
}
// Instruction descriptor of kind::f16: f32 accumulator (bits 4-5 = 1), bf16 A and B (bits 7-9, 10-12 = 1),
// B major in bit 16 (0 = K-major, 1 = MN-major), N / 8 in bits 17-22, M / 16 in bits 24-28.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, bool b_mn_major, bool f16 = false) {
    return (1u << 4) | ((f16 ? 0u : 1u) << 7) | ((f16 ? 0u : 1u) << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);       // (A / B format fields: 0 = f16, 1 = bf16)
}
// Packed pairs of f32 (two lanes of one 64-bit register): one instruction for two multiply-adds / adds.
__device__ __forceinline__ uint64_t f2_pack(float x, float y) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(d) : "f"(x), "f"(y));
    return d;
}
__device__ __forceinline__ void f2_unpack(uint64_t d, float &x, float &y) { asm("mov.b64 {%0, %1}, %2;\n" : "=f"(x), "=f"(y) : "l"(d)); }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^t for a pair of arguments without the special-function unit: t = n + f with n the nearest integer (magic-number
// rounding), 2^f by a cubic on [-1/2, 1/2] (relative error 7.5e-5, far below the bf16 rounding of the weights that
// follows), 2^n by adding n to the exponent field.  Arguments are clamped at -126 (the result is then ~1e-38, i.e. 0
// for a softmax weight); the caller guarantees t <= 8 + log2(64).
__device__ __forceinline__ void exp2_pair_fma(float t0, float t1, float &e0, float &e1) {
    const float kMagic = 12582912.f;                         // 1.5 * 2^23: adding it rounds to the nearest integer
    t0 = fmaxf(t0, -126.f);
    t1 = fmaxf(t1, -126.f);
    const uint64_t t2 = f2_pack(t0, t1);
    const uint64_t r2 = f2_add(t2, f2_pack(kMagic, kMagic));
    const uint64_t n2 = f2_add(r2, f2_pack(-kMagic, -kMagic));
    const uint64_t f2 = f2_fma(n2, f2_pack(-1.f, -1.f), t2);
    uint64_t p2 = f2_fma(f2, f2_pack(0.0551716648f, 0.0551716648f), f2_pack(0.2426111251f, 0.2426111251f));
    p2 = f2_fma(p2, f2, f2_pack(0.6932609677f, 0.6932609677f));
    p2 = f2_fma(p2, f2, f2_pack(0.9999280572f, 0.9999280572f));
    float r0, r1, p0, p1;
    f2_unpack(r2, r0, r1);
    f2_unpack(p2, p0, p1);
    e0 = __uint_as_float(__float_as_uint(r0) * 0x00800000u + __float_as_uint(p0));   // low mantissa bits of r hold n
    e1 = __uint_as_float(__float_as_uint(r1) * 0x00800000u + __float_as_uint(p1));
}
#ifndef GVA_PREFILL_EMU_EVERY
#define GVA_PREFILL_EMU_EVERY 0     // build-time knob: every n-th pair of exponentials runs on the FMA pipe (0 = none;
                                    // measured slower at 4, 3 and 2: the XU pipe is not what the warps wait for)
#endif
constexpr float kRescaleLog2 = 8.f;   // the softmax reference moves only when the running maximum grows by more than 2^8
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// Bounded wait for the softmax warps, whose barriers are normally complete already: a bare poll first.
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_bounded(bar, parity, abort_flag);
}
// Bounded wait whose polls sleep in hardware (suspend-time hint) instead of spinning through the issue slots.
__device__ __forceinline__ bool mbar_wait_sleepy(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        __nanosleep(64);
        if ((it & 7u) == 7u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) return false;
        }
    }
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;\n" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// the pair (x, y) as 16-bit floats of the kernel's operand type: bf16, or f16 over the 8-bit cache
template <bool F16>
__device__ __forceinline__ uint32_t pack_op(float x, float y) { return F16 ? pack_f16(x, y) : pack_bf16(x, y); }
// ... and back to f32 (low, high element)
template <bool F16>
__device__ __forceinline__ void unpack_op(uint32_t w, float &x, float &y) {
    if constexpr (F16) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
        x = f.x;
        y = f.y;
    } else {
        x = __uint_as_float(w << 16);
        y = __uint_as_float(w & 0xffff0000u);
    }
}

template <int DV, int DR, bool C8 = false>
__global__ void __launch_bounds__(192, PrefillTraits<DV, DR, C8>::BLOCKS_PER_SM)
prefill_kernel(PrefillParams p, const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_k) {
    using T = PrefillTraits<DV, DR, C8>;
    constexpr int NS = T::NSTAGE;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.z, g = blockIdx.y;
    const int S = p.num_splits, split = blockIdx.x % S;
    const int qb = gridDim.x / S - 1 - blockIdx.x / S;   // the longest rows (last query blocks) are scheduled first
    grid_dependency_wait();
    const int q_begin = p.cu_q[b];
    const int n_q = p.cu_q[b + 1] - q_begin;
    const int q0 = qb * T::QTOK;
    if (q0 >= n_q) return;
    const int ctx = p.ctx_lens[b];
    const long long kv_total = (long long)ctx + n_q;   // tokens of this sequence in the cache (context + chunk)
    if (ctx < 0 || kv_total > (long long)p.max_pages * p.P) {
        if (tid == 0) report_error(p.dev_status, GVA_ERR_SEQ_LEN, b);
        return;
    }
    const int nv = min(T::QTOK, n_q - q0);             // live query tokens of this block
    const int p0 = ctx + q0;                           // position of the block's first query token
    const int n_all = (p0 + nv - 1) / T::TILE + 1;     // tiles 0..n_all-1 hold every visible token
    const int per_split = (n_all + S - 1) / S;
    const int t_lo = split * per_split;                // this block's tiles: t_lo .. t_lo + n_tiles - 1 (tile j below is local)
    const int n_tiles = min(n_all, t_lo + per_split) - t_lo;
    if (n_tiles <= 0) {                                // more splits than tiles: an empty range weighs nothing in the merge
        if (tid < T::ROWS && (tid >> 2) < nv) {
            float *ml = p.part_ml + (((size_t)(q_begin + q0 + (tid >> 2)) * p.H + g * kHeadsPerGroup + (tid & 3)) * S + split) * 2;
            ml[0] = -INFINITY;
            ml[1] = 0.f;
        }
        return;
    }

    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + T::OFF_BAR);
    const uint32_t bar0 = s_base + T::OFF_BAR;
    auto kv_full = [&](int s) { return bar0 + 8u * s; };
    auto kv_empty = [&](int s) { return bar0 + 8u * (NS + s); };
    auto s_full = [&](int i) { return bar0 + 8u * (2 * NS + i); };
    // one P barrier per score buffer: the softmax of tile j+1 can end before the value-product issuer has observed tile j,
    // and a single barrier waited on by parity would then be two phases ahead of its waiter
    auto p_full = [&](int i) { return bar0 + 8u * (2 * NS + ((i & 1) ? 8 : 3)); };
    const uint32_t q_ready = bar0 + 8u * (2 * NS + 4), drain = bar0 + 8u * (2 * NS + 5),
                   o_full = bar0 + 8u * (2 * NS + 6), drain2 = bar0 + 8u * (2 * NS + 7);
    auto raw_full = [&](int s) { return bar0 + 8u * (2 * NS + 9 + s); };     // 8-bit cache: the byte tiles of a stage have landed
    constexpr int NB = T::NSBUF;
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(bars + T::N_BARS);
    volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(kv_full(s), C8 ? T::ROWS : 1);      // (8-bit cache: one arrival per softmax thread that widened its share)
            mbar_init(kv_empty(s), 1);
        }
        mbar_init(s_full(0), 1);
        mbar_init(s_full(1), 1);
        mbar_init(s_full(2), 1);
        mbar_init(p_full(0), T::ROWS);
        mbar_init(p_full(1), T::ROWS);
        mbar_init(q_ready, T::ROWS);
        mbar_init(drain, 1);
        mbar_init(drain2, 1);
        mbar_init(o_full, 1);
        if constexpr (C8)
            for (int s = 0; s < NS; ++s) mbar_init(raw_full(s), 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
    }
    if (warp == 5) {
        tmem_alloc(smem_u32(s_tmem), T::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;

    if (warp < 4) {
        // ====================================== softmax: one row per thread ======================================
        const int r = tid;
        const int tok = r >> 2, hl = r & 3;
        const int h = g * kHeadsPerGroup + hl;
        const bool live = tok < nv;
        const int pos = p0 + tok;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        // ---- stage Q as bf16: into tensor memory (row = lane, two values per column) or, where that does not fit,
        //      into shared memory as swizzled K-major rows (value dims in 128-byte boxes, then the RoPE dims) ----
        {
            // q = hi + lo with hi = bf16(q), lo = bf16(q - hi): the score product is taken with both, so the absorbed
            // query enters with ~16 significant bits and a score of any size is as exact as the cache's own bf16 values
            // allow (with hi alone a score s is off by about |s| 2^-9, which is what limits accuracy on peaked rows).
            const float4 *src = reinterpret_cast<const float4 *>(p.q_abs + ((size_t)(q_begin + q0 + tok) * p.H + h) * (DV + DR));
            auto split4 = [](const float4 &a, uint32_t &h01, uint32_t &h23, uint32_t &l01, uint32_t &l23) {
                float b0, b1, b2, b3;
                h01 = pack_op<C8>(a.x, a.y);
                h23 = pack_op<C8>(a.z, a.w);
                unpack_op<C8>(h01, b0, b1);
                unpack_op<C8>(h23, b2, b3);
                l01 = pack_op<C8>(a.x - b0, a.y - b1);
                l23 = pack_op<C8>(a.z - b2, a.w - b3);
            };
            // value dims: 16-byte piece c (8 values) of the row, as swizzled K-major rows in 128-byte boxes; then the RoPE dims
#pragma unroll
            for (int c = 0; c < DV / 8; ++c) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), bq = a;
                if (live) {
                    a = __ldg(src + 2 * c);
                    bq = __ldg(src + 2 * c + 1);
                }
                uint32_t hw[4], lw[4];
                split4(a, hw[0], hw[1], lw[0], lw[1]);
                split4(bq, hw[2], hw[3], lw[2], lw[3]);
                const uint32_t off = (c >> 3) * T::QBOX_BYTES + swz128(r, c & 7);
                if constexpr (!T::LO_IN_TMEM) *reinterpret_cast<uint4 *>(smem + T::OFF_LOV + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                else tmem_st4_nowait(lane_base + T::COL_QLO + c * 4, lw);
                if constexpr (!T::Q_IN_TMEM) *reinterpret_cast<uint4 *>(smem + T::OFF_QV + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                else tmem_st4_nowait(lane_base + T::COL_Q + c * 4, hw);
            }
#pragma unroll
            for (int c = 0; c < T::DRP / 8; ++c) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), bq = a;
                if (live && c * 8 < DR) {
                    a = __ldg(src + DV / 4 + 2 * c);
                    bq = __ldg(src + DV / 4 + 2 * c + 1);
                }
                uint32_t hw[4], lw[4];
                split4(a, hw[0], hw[1], lw[0], lw[1]);
                split4(bq, hw[2], hw[3], lw[2], lw[3]);
                const uint32_t off = swz_kr<T::KR_ROW>(r, c);
                if constexpr (!T::LO_IN_TMEM) *reinterpret_cast<uint4 *>(smem + T::OFF_LOR + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                else tmem_st4_nowait(lane_base + T::COL_QLO + DV / 2 + c * 4, lw);
                if constexpr (!T::Q_IN_TMEM) *reinterpret_cast<uint4 *>(smem + T::OFF_QR + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                else tmem_st4_nowait(lane_base + T::COL_Q + DV / 2 + c * 4, hw);
            }
            if constexpr (T::Q_IN_TMEM) {
                tmem_st_wait();
                tc_fence_before();
            }
            fence_async_smem();
            mbar_arrive(q_ready);
        }

        float m_run = -INFINITY, l_run = 0.f;          // softmax reference (log2 domain) and sum relative to it
        const uint32_t o_addr = lane_base + T::COL_O;
        bool ok = true;
        // 8-bit cache: the 128 softmax threads widen a tile's e4m3 codes to f16 (exact) from the stage's raw region into its
        // swizzled operand tiles, 16 codes in and two 16-byte pieces out per step, two or three steps per thread and tile; rows
        // at or beyond the end of the cache become zeros.  Tile t + 2 is widened at the top of iteration t -- its score
        // product cannot start before the value product of tile t has released the score buffer -- so the widening is
        // never on the chain of dependent steps.  (Its stage was refilled only after the value product of tile t + 2 - NS.)
        auto convert_tile = [&](int t) -> bool {
            const int st = t % NS;
            if (!__all_sync(0xffffffffu, mbar_wait_spin(raw_full(st), (t / NS) & 1, s_abort))) return false;
            unsigned char *stage = smem + T::OFF_STAGE + st * T::STAGE_BYTES;
            const unsigned char *raw = stage + T::OFF_RAW;
            const long long tok0 = (long long)(t_lo + t) * T::TILE;
            constexpr int NPV = T::TILE * (DV / 16) / T::ROWS;      // 16-byte pieces of the value tile per thread
            uint4 xv[NPV], xk = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < NPV; ++u) {                         // all loads first: one shared-memory round trip
                const int pc = tid + T::ROWS * u;
                xv[u] = *reinterpret_cast<const uint4 *>(raw + (pc / (DV / 16)) * DV + (pc % (DV / 16)) * 16);
            }
            constexpr int NPK = T::TILE * (DR / 16);                // pieces of the positional tile (at most one per thread)
            static_assert(NPK <= T::ROWS, "one positional piece per thread at most");
            if (DR > 0 && tid < NPK) xk = *reinterpret_cast<const uint4 *>(raw + T::RAW_V_BYTES + tid * 16);
#pragma unroll
            for (int u = 0; u < NPV; ++u) {
                const int pc = tid + T::ROWS * u;
                const int r = pc / (DV / 16), c16 = pc % (DV / 16);
                uint4 x = xv[u];
                if (tok0 + r >= kv_total) x = make_uint4(0, 0, 0, 0);
                uint4 lo4, hi4;
                e4m3x4_to_f16x2(x.x, lo4.x, lo4.y);
                e4m3x4_to_f16x2(x.y, lo4.z, lo4.w);
                e4m3x4_to_f16x2(x.z, hi4.x, hi4.y);
                e4m3x4_to_f16x2(x.w, hi4.z, hi4.w);
                unsigned char *box = stage + (c16 / 4) * T::VBOX_BYTES;
                const int c = (c16 % 4) * 2;
                *reinterpret_cast<uint4 *>(box + swz128(r, c)) = lo4;
                *reinterpret_cast<uint4 *>(box + swz128(r, c + 1)) = hi4;
            }
            if (DR > 0 && tid < NPK) {
                const int r = tid / (DR > 0 ? DR / 16 : 1), c16 = tid % (DR > 0 ? DR / 16 : 1);
                uint4 lo4, hi4;
                e4m3x4_to_f16x2(xk.x, lo4.x, lo4.y);
                e4m3x4_to_f16x2(xk.y, lo4.z, lo4.w);
                e4m3x4_to_f16x2(xk.z, hi4.x, hi4.y);
                e4m3x4_to_f16x2(xk.w, hi4.z, hi4.w);
                *reinterpret_cast<uint4 *>(stage + T::V_BYTES + swz_kr<T::KR_ROW>(r, 2 * c16)) = lo4;
                *reinterpret_cast<uint4 *>(stage + T::V_BYTES + swz_kr<T::KR_ROW>(r, 2 * c16 + 1)) = hi4;
            }
            fence_async_smem();      // generic-proxy writes before the tensor core's reads
            mbar_arrive(kv_full(st));
            return true;
        };
        if constexpr (C8) {
            for (int t = 0; t < 2 && t < n_tiles && ok; ++t) ok = convert_tile(t);
        }
        // A warp none of whose 8 query tokens is live (short chunks, multi-token decode) only keeps the barrier protocol
        // going: its rows of S, P and O are never used.  (S of tile j complete implies the P barrier of tile j-2 has
        // completed, so an arrival for tile j cannot fall into an earlier phase.)
        const bool warp_dead = warp * 8 >= nv;
        for (int j = 0; j < n_tiles && ok; ++j) {
            if constexpr (C8) {
                if (j + 2 < n_tiles && !convert_tile(j + 2)) { ok = false; break; }
            }
            if (!__all_sync(0xffffffffu, mbar_wait_spin(s_full(j % NB), (j / NB) & 1, s_abort))) { ok = false; break; }   // warp-uniform
            // rows of the last tile at or beyond the end of the cache may hold anything (NaN): zero them, P = 0 there
            // (the score product of this tile has completed, the value product starts only after the arrivals below)
            if (!C8 && (long long)(t_lo + j + 1) * T::TILE > kv_total) {      // (the 8-bit path zeroes them while it widens the tile)
                if (tid < T::TILE && (long long)(t_lo + j) * T::TILE + tid >= kv_total) {
                    unsigned char *vrow = smem + T::OFF_STAGE + (j % NS) * T::STAGE_BYTES;
#pragma unroll
                    for (int bx = 0; bx < T::BOXES; ++bx)
#pragma unroll
                        for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4 *>(vrow + bx * T::VBOX_BYTES + tid * 128 + c * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_async_smem();
            }
            if (warp_dead) {
                mbar_arrive(p_full(j));
                continue;
            }
            tc_fence_after();
            const uint32_t s_addr = lane_base + T::COL_S + (j % NB) * T::TILE;
            float s[T::TILE];
            {
                float lo[32], hi[32];
                tmem_ld32_nowait(s_addr, lo);
                tmem_ld32_nowait(s_addr + 32, hi);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; ++c) { s[c] = lo[c]; s[32 + c] = hi[c]; }
            }
            const int limit = pos - (t_lo + j) * T::TILE;     // columns c > limit are in the future of this row
            if (limit < T::TILE - 1) {
#pragma unroll
                for (int c = 0; c < T::TILE; ++c) s[c] = (c > limit) ? -INFINITY : s[c];
            }
            uint32_t pk[T::TILE / 2];
            float tile_sum = 0.f;
            // weights and their sum relative to the reference m_ref; P as bf16 pairs
            auto weights = [&](float m_ref) {
                const float nm = (m_ref == -INFINITY) ? 0.f : -m_ref;   // a row that has seen nothing yet: all weights 0, not NaN
                const uint64_t sc2 = f2_pack(p.scale_log2, p.scale_log2), nm2 = f2_pack(nm, nm);
                uint64_t sum2[2] = {f2_pack(0.f, 0.f), f2_pack(0.f, 0.f)};
#pragma unroll
                for (int c = 0; c < T::TILE; c += 2) {
                    float t0, t1, e0, e1;
                    f2_unpack(f2_fma(f2_pack(s[c], s[c + 1]), sc2, nm2), t0, t1);
                    if (GVA_PREFILL_EMU_EVERY > 0 && ((c >> 1) % (GVA_PREFILL_EMU_EVERY > 0 ? GVA_PREFILL_EMU_EVERY : 1)) == 1) {
                        exp2_pair_fma(t0, t1, e0, e1);       // a share of the exponentials can bypass the XU pipe
                    } else {
                        e0 = fast_exp2(t0);
                        e1 = fast_exp2(t1);
                    }
                    sum2[(c >> 1) & 1] = f2_add(sum2[(c >> 1) & 1], f2_pack(e0, e1));
                    pk[c >> 1] = pack_op<C8>(e0, e1);
                }
                float sa, sb;
                f2_unpack(f2_add(sum2[0], sum2[1]), sa, sb);
                tile_sum = sa + sb;
            };
            // From the second tile on the weights are computed against the current reference at once, while the row
            // maximum is still being reduced (the two instruction streams are independent); the rare tile whose
            // maximum moves the reference is redone.
            if (j > 0) weights(m_run);
            float mx[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) mx[k] = max3(s[k], s[k + 4], s[k + 8]);
#pragma unroll
            for (int c = 12; c + 8 <= T::TILE; c += 8)
#pragma unroll
                for (int k = 0; k < 4; ++k) mx[k] = max3(mx[k], s[c + k], s[c + 4 + k]);
#pragma unroll
            for (int k = 0; k < 4; ++k) mx[k] = fmaxf(mx[k], s[T::TILE - 4 + k]);
            const float m_tile = max3(mx[0], mx[1], fmaxf(mx[2], mx[3])) * p.scale_log2;
            // The reference m_run of the row only moves when the tile's maximum exceeds it by more than 2^8: the
            // weights stay below 256 relative to it, the result is the same quotient, and the accumulated O (which
            // lives in tensor memory) has to be rescaled only then.  (Token 0 is visible to every row, so m_tile is
            // finite in global tile 0; a later split can start with tiles a row does not see at all: its reference
            // stays -inf and its weights are 0 until it sees something.)
            const bool move = m_tile > m_run + kRescaleLog2;
            // tcgen05.ld / tcgen05.st are warp-wide instructions: when any row of the warp moves its reference, every
            // lane rescales its row of O (by 1 where nothing moved), once the value product of tile j-1 has landed
            if (j == 0 || __any_sync(0xffffffffu, move)) {
                float alpha = 1.f;
                if (move) {
                    alpha = fast_exp2(m_run - m_tile);
                    l_run *= alpha;
                    m_run = m_tile;
                }
                if (j > 0) {
                    if (!__all_sync(0xffffffffu, mbar_wait_spin(kv_empty((j - 1) % NS), ((j - 1) / NS) & 1, s_abort))) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t al2 = f2_pack(alpha, alpha);
#pragma unroll
                    for (int part = 0; part < DV / 32; ++part) {
                        float o[32];
                        tmem_ld32_nowait(o_addr + part * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; i += 2) f2_unpack(f2_mul(f2_pack(o[i], o[i + 1]), al2), o[i], o[i + 1]);
                        tmem_st32(o_addr + part * 32, o);
                    }
                }
                weights(m_run);
            }
            // P goes over the first 32 columns of this tile's S (the row's only reader is this thread)
            tmem_st32u_nowait(s_addr, pk);
            l_run += tile_sum;
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(p_full(j));
        }
        if (ok && !__all_sync(0xffffffffu, mbar_wait_spin(o_full, 0, s_abort))) ok = false;
        if (ok && !warp_dead) {
            tc_fence_after();
            // (tcgen05.ld is a warp-wide instruction: every lane takes part, dead rows only skip the stores)
            const size_t row_h = (size_t)(q_begin + q0 + tok) * p.H + h;
            const bool whole = S == 1;
            const float inv = whole ? 1.f / l_run : 1.f;          // a split leaves O unnormalised for the merge
            float *dst = whole ? p.out + row_h * DV : p.part_o + (row_h * S + split) * DV;
#pragma unroll
            for (int part = 0; part < DV / 32; ++part) {
                float o[32];
                tmem_ld32_nowait(o_addr + part * 32, o);
                tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4 *>(dst + part * 32 + i) = make_float4(o[i] * inv, o[i + 1] * inv, o[i + 2] * inv, o[i + 3] * inv);
                }
            }
            if (live) {
                if (whole) {
                    if (p.lse) p.lse[row_h] = (m_run + log2f(l_run)) * kLn2;
                } else {
                    p.part_ml[(row_h * S + split) * 2] = m_run;
                    p.part_ml[(row_h * S + split) * 2 + 1] = l_run;
                }
            }
        } else if (!ok && !*s_abort) {
            report_error(p.dev_status, GVA_ERR_TIMEOUT, b);
            *s_abort = 1;
        }
        tc_fence_before();
    } else {
        // ========== MMA issuers: warp 5 the score products, warp 4 the value products (and the TMA loads) ==========
        // One thread sustains about one tcgen05.mma per 110 cycles (measured), and a 128 x 64 x 16 MMA occupies the tensor
        // pipe for 32: two issuing threads per block (and two blocks per SM) are needed to keep the pipe fed.
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc(T::ROWS, T::TILE, false, C8);
            constexpr uint32_t idesc_o = umma_idesc(T::ROWS, DV, true, C8);
            constexpr uint64_t kr_swz = T::KR_ROW == 32 ? kSwz32 : kSwz64;
            constexpr uint32_t kr_sbo = 8 * T::KR_ROW;
            // Descriptors differ only in their 14-bit start-address field (low word): the high words and the other low
            // bits are compile-time constants, so one issue costs an add per operand, not a descriptor build.
            constexpr uint32_t hi128 = (1024u >> 4) | (1u << 14) | ((uint32_t)kSwz128 << 29);      // SBO 1024, version 1, 128-byte swizzle
            constexpr uint32_t hikr = (kr_sbo >> 4) | (1u << 14) | ((uint32_t)kr_swz << 29);
            constexpr uint32_t lo_k = (16u >> 4) << 16;                                           // LBO 16 (K-major operands)
            constexpr uint32_t lo_mn = ((uint32_t)T::VBOX_BYTES >> 4) << 16;                      // LBO = box stride (MN-major value tile)
            const uint32_t a_qv = ((s_base + T::OFF_QV) & 0x3FFFFu) >> 4, a_qr = ((s_base + T::OFF_QR) & 0x3FFFFu) >> 4;
            const uint32_t a_lov = ((s_base + T::OFF_LOV) & 0x3FFFFu) >> 4, a_lor = ((s_base + T::OFF_LOR) & 0x3FFFFu) >> 4;
            const uint32_t a_st = ((s_base + T::OFF_STAGE) & 0x3FFFFu) >> 4;
            auto mk = [](uint32_t lo, uint32_t hi) { return (uint64_t)lo | ((uint64_t)hi << 32); };
            constexpr int KS_S = T::KSTEPS_V + T::KSTEPS_R, KS_O = T::TILE / 16;
            bool ok = true;
            int issued_mma = 0;
            if (warp == 5) {
                ok = mbar_wait_spin(q_ready, 0, s_abort);
                for (int t = 0; t < n_tiles && ok; ++t) {
                    // S[t & 1] also holds the P of tile t-2, so the value product of that tile must have completed before the
                    // score product of tile t is issued (MMAs with different accumulators are not ordered among themselves)
                    if (!mbar_wait_spin(kv_full(t % NS), (t / NS) & 1, s_abort)) { ok = false; break; }
                    if (t >= NB && !mbar_wait_spin(kv_empty((t - NB) % NS), ((t - NB) / NS) & 1, s_abort)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t vb = a_st + (uint32_t)(t % NS) * (T::STAGE_BYTES >> 4);
                    const uint32_t d = tmem + T::COL_S + (t % NB) * T::TILE;
#pragma unroll
                    for (int ks = 0; ks < KS_S; ++ks) {
                        if (ks < T::KSTEPS_V) {
                            const uint32_t off = ((ks >> 2) * T::QBOX_BYTES + (ks & 3) * 32) >> 4;
                            const uint32_t voff = ((ks >> 2) * T::VBOX_BYTES + (ks & 3) * 32) >> 4;
                            if constexpr (T::Q_IN_TMEM) umma_bf16_ts(d, tmem + T::COL_Q + ks * 8, mk((vb + voff) | lo_k, hi128), idesc_s, ks > 0);
                            else umma_bf16(d, mk((a_qv + off) | lo_k, hi128), mk((vb + voff) | lo_k, hi128), idesc_s, ks > 0);
                        } else {
                            const uint32_t kr = (uint32_t)(ks - T::KSTEPS_V) * 2;
                            if constexpr (T::Q_IN_TMEM) umma_bf16_ts(d, tmem + T::COL_Q + ks * 8, mk((vb + (T::V_BYTES >> 4) + kr) | lo_k, hikr), idesc_s, 1);
                            else umma_bf16(d, mk((a_qr + kr) | lo_k, hikr), mk((vb + (T::V_BYTES >> 4) + kr) | lo_k, hikr), idesc_s, 1);
                        }
                    }
                    // ... and the same k-steps again with the low-order halves of the query
#pragma unroll
                    for (int ks = 0; ks < KS_S; ++ks) {
                        if (ks < T::KSTEPS_V) {
                            const uint32_t off = ((ks >> 2) * T::QBOX_BYTES + (ks & 3) * 32) >> 4;
                            const uint32_t voff = ((ks >> 2) * T::VBOX_BYTES + (ks & 3) * 32) >> 4;
                            if constexpr (T::LO_IN_TMEM) umma_bf16_ts(d, tmem + T::COL_QLO + ks * 8, mk((vb + voff) | lo_k, hi128), idesc_s, 1);
                            else umma_bf16(d, mk((a_lov + off) | lo_k, hi128), mk((vb + voff) | lo_k, hi128), idesc_s, 1);
                        } else {
                            const uint32_t kr = (uint32_t)(ks - T::KSTEPS_V) * 2;
                            if constexpr (T::LO_IN_TMEM) umma_bf16_ts(d, tmem + T::COL_QLO + ks * 8, mk((vb + (T::V_BYTES >> 4) + kr) | lo_k, hikr), idesc_s, 1);
                            else umma_bf16(d, mk((a_lor + kr) | lo_k, hikr), mk((vb + (T::V_BYTES >> 4) + kr) | lo_k, hikr), idesc_s, 1);
                        }
                    }
                    umma_commit(s_full(t % NB));
                    ++issued_mma;
                }
            } else {
                // This thread is also the producer: it fills the ring first, and after each value product it refills the
                // stage that the previous value product has released.
                int loaded = 0;
                auto load_tile = [&](int t) -> bool {
                    const int st = t % NS;
                    const int t0 = (t_lo + t) * T::TILE;
                    const int pj = t0 / p.P, slot0 = t0 % p.P;
                    const long long page = p.block_table ? (long long)p.block_table[(size_t)b * p.max_pages + pj]
                                                         : (long long)b * p.max_pages + pj;
                    if (page < 0 || page >= p.num_pages) {
                        report_error(p.dev_status, GVA_ERR_BAD_PAGE, b);
                        *s_abort = 1;
                        return false;
                    }
                    const uint32_t dst = s_base + T::OFF_STAGE + st * T::STAGE_BYTES;
                    const int row = (int)((page * p.G + g) * p.P + slot0);
                    if constexpr (C8) {      // byte tiles into the stage's raw region; the softmax warps widen them
                        mbar_expect_tx(raw_full(st), T::RAW_V_BYTES + T::RAW_K_BYTES);
                        tma_load_2d(dst + T::OFF_RAW, &tm_v, 0, row, raw_full(st));
                        if constexpr (DR > 0) tma_load_2d(dst + T::OFF_RAW + T::RAW_V_BYTES, &tm_k, 0, (int)(page * p.P + slot0), raw_full(st));
                    } else {
                        mbar_expect_tx(kv_full(st), T::V_BYTES + T::KR_BYTES);
#pragma unroll
                        for (int bx = 0; bx < T::BOXES; ++bx) tma_load_2d(dst + bx * T::VBOX_BYTES, &tm_v, bx * 64, row, kv_full(st));
                        if constexpr (DR > 0) tma_load_2d(dst + T::V_BYTES, &tm_k, 0, (int)(page * p.P + slot0), kv_full(st));   // (no positional tile in a value-only cache)
                    }
                    ++loaded;
                    return true;
                };
                for (int t = 0; t < NS && t < n_tiles && ok; ++t) ok = load_tile(t);
                for (int j = 0; j < n_tiles && ok; ++j) {
                    // every row has stored P of tile j and finished any rescaling of O
                    if (!mbar_wait_spin(p_full(j), (j >> 1) & 1, s_abort)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t vb = a_st + (uint32_t)(j % NS) * (T::STAGE_BYTES >> 4);
#pragma unroll
                    for (int ks = 0; ks < KS_O; ++ks)
                        umma_bf16_ts(tmem + T::COL_O, tmem + T::COL_S + (j % NB) * T::TILE + ks * 8,
                                     mk((vb + ks * (16 * 128 >> 4)) | lo_mn, hi128), idesc_o, (j > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(kv_empty(j % NS));
                    ++issued_mma;
                    if (j >= 1 && j - 1 + NS < n_tiles) {      // tile j-1 was consumed a tile ago: its stage takes tile j-1+NS
                        if (!mbar_wait_spin(kv_empty((j - 1) % NS), ((j - 1) / NS) & 1, s_abort)) { ok = false; break; }
                        ok = load_tile(j - 1 + NS);
                    }
                }
                if (ok) umma_commit(o_full);
                if (*s_abort) {   // copies still in flight must land before the block's shared memory is released
                    for (int t = max(0, loaded - NS); t < loaded; ++t)
                        for (int it = 0; it < kDrainPolls && !mbar_try_wait(C8 ? raw_full(t % NS) : kv_full(t % NS), (t / NS) & 1); ++it) {}
                }
            }
            if (!ok && !*s_abort) {
                report_error(p.dev_status, GVA_ERR_TIMEOUT, b);
                *s_abort = 1;
            }
            // nothing issued by this thread may still be running (or about to signal a barrier) when the block ends
            if (issued_mma > 0) {
                const uint32_t dr = warp == 5 ? drain : drain2;
                umma_commit(dr);
                for (int it = 0; it < kDrainPolls * 16 && !mbar_try_wait(dr, 0); ++it) {}
            }
            tc_fence_before();
        }
    }
    grid_dependency_launch();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem, T::TMEM_COLS);
    }
}

// ---- merge of split-KV partial results: one warp per (query row, head) -----------------------------------
template <int DV>
__global__ void __launch_bounds__(128)
merge_splits_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml, float *__restrict__ out,
                    float *__restrict__ lse, int rows, int S) {
    grid_dependency_launch();
    grid_dependency_wait();
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float *ml = part_ml + (size_t)row * S * 2;
    float m_max = -INFINITY;
    for (int s = 0; s < S; ++s) m_max = fmaxf(m_max, ml[2 * s]);
    float acc[DV / 32];
#pragma unroll
    for (int i = 0; i < DV / 32; ++i) acc[i] = 0.f;
    float L = 0.f;
    for (int s = 0; s < S; ++s) {
        const float l = ml[2 * s + 1];
        if (!(l > 0.f)) continue;                      // an empty range left its O unwritten
        const float w = fast_exp2(ml[2 * s] - m_max);
        L += w * l;
        const float *o = part_o + ((size_t)row * S + s) * DV;
#pragma unroll
        for (int i = 0; i < DV / 32; ++i) acc[i] = fmaf(w, o[i * 32 + lane], acc[i]);
    }
    const float inv = 1.f / L;
#pragma unroll
    for (int i = 0; i < DV / 32; ++i) out[(size_t)row * DV + i * 32 + lane] = acc[i] * inv;
    if (lse && lane == 0) lse[row] = (m_max + log2f(L)) * kLn2;
}

// ---- host: support check, tensor maps, launch ---------------------------------------------------------
inline bool prefill_supported(const gva_config &cfg) {
    if (cfg.cache_dtype == GVA_E4M3 && cfg.d_r == 24) return false;
    return (cfg.cache_dtype == GVA_BF16 || cfg.cache_dtype == GVA_E4M3) && cfg.page_size % 64 == 0 && cfg.H / cfg.G == kHeadsPerGroup &&
           ((cfg.d_v == 64 && (cfg.d_r == 16 || cfg.d_r == 24 || cfg.d_r == 0)) || (cfg.d_v == 128 && (cfg.d_r == 32 || cfg.d_r == 0)));
}

template <int DV, int DR, bool C8 = false>
int launch_prefill_t(const gva_config &cfg, const MmaHostState &st, int smem_optin, const PrefillParams &p, const void *v_pool,
                     const void *kr_pool, int B, int max_q_len, int n_q, cudaStream_t stream) {
    using T = PrefillTraits<DV, DR, C8>;
    // never more blocks on an SM than its 512 tensor-memory columns can serve: pad the request if need be
    const size_t floor_bytes = (size_t)227 * 1024 / (T::BLOCKS_PER_SM + 1) + 1024;
    const size_t smem = (size_t)T::SMEM_BYTES < floor_bytes ? floor_bytes : (size_t)T::SMEM_BYTES;
    if (smem > (size_t)smem_optin) return GVA_ERR_UNSUPPORTED;
    auto fn = prefill_kernel<DV, DR, C8>;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GVA_ERR_CUDA;
    CUtensorMap tm_v, tm_k;
    if constexpr (C8) {       // byte tiles, unswizzled: rows of d_v and of d_r codes
        if (!encode_map_u8(st, &tm_v, v_pool, DV, (uint64_t)p.num_pages * cfg.G * p.P, DV, T::TILE, CU_TENSOR_MAP_SWIZZLE_NONE))
            return GVA_ERR_CUDA;
        if (DR == 0) tm_k = tm_v;
        else if (!encode_map_u8(st, &tm_k, kr_pool, DR, (uint64_t)p.num_pages * p.P, DR, T::TILE, CU_TENSOR_MAP_SWIZZLE_NONE))
            return GVA_ERR_CUDA;
    } else if (!encode_map(st, &tm_v, v_pool, DV, (uint64_t)p.num_pages * cfg.G * p.P, 64, T::TILE, CU_TENSOR_MAP_SWIZZLE_128B)) {
        return GVA_ERR_CUDA;
    } else if (DR == 0) {
        tm_k = tm_v;      // value-only cache: there is no positional-key tile to describe (the kernel never uses this map)
    } else if (!encode_map(st, &tm_k, kr_pool, DR, (uint64_t)p.num_pages * p.P, DR > 0 ? T::DRP : 16, T::TILE,
                           T::DRP == 16 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_64B)) {
        return GVA_ERR_CUDA;
    }
    const dim3 grid(((max_q_len + T::QTOK - 1) / T::QTOK) * p.num_splits, cfg.G, B);
    if (launch_pdl(fn, grid, dim3(T::THREADS), smem, stream, p, tm_v, tm_k) != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    if (p.num_splits > 1) {
        const int rows = n_q * cfg.H;
        if (launch_pdl(merge_splits_kernel<DV>, dim3((rows + 3) / 4), dim3(128), 0, stream, (const float *)p.part_o,
                       (const float *)p.part_ml, p.out, p.lse, rows, p.num_splits) != cudaSuccess) {
            (void)cudaGetLastError();
            return GVA_ERR_CUDA;
        }
    }
    return GVA_OK;
}

inline int launch_prefill(const gva_config &cfg, const MmaHostState &st, int smem_optin, const PrefillParams &p,
                          const void *v_pool, const void *kr_pool, int B, int max_q_len, int n_q, cudaStream_t stream) {
    if (!prefill_supported(cfg)) return GVA_ERR_UNSUPPORTED;
    if ((uint64_t)p.num_pages * cfg.G * cfg.page_size >= (1ull << 31)) return GVA_ERR_UNSUPPORTED;
    if (cfg.cache_dtype == GVA_E4M3) {
        if (cfg.d_v == 64)
            return cfg.d_r == 16 ? launch_prefill_t<64, 16, true>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream)
                                 : launch_prefill_t<64, 0, true>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
        return cfg.d_r == 32 ? launch_prefill_t<128, 32, true>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream)
                             : launch_prefill_t<128, 0, true>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
    }
    if (cfg.d_r == 0) {       // value-only cache
        if (cfg.d_v == 64) return launch_prefill_t<64, 0>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
        return launch_prefill_t<128, 0>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
    }
    if (cfg.d_v == 64 && cfg.d_r == 24) return launch_prefill_t<64, 24>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
    if (cfg.d_v == 64) return launch_prefill_t<64, 16>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
    return launch_prefill_t<128, 32>(cfg, st, smem_optin, p, v_pool, kr_pool, B, max_q_len, n_q, stream);
}

}  // namespace gva
