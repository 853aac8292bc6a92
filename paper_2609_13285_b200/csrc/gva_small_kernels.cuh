// The O(1)-in-T kernels of a decode step: query absorption (Eq. absorb + query-side RoPE), cache
// append (Algorithm 1's append lines) and the log-sum-exp merge of split-KV partial results.
#pragma once

#include <type_traits>

#include "gva_common.cuh"

namespace gva {

constexpr int kMaxRopePairs = 16;   // d_r <= 32

struct RopeTable {
    double inv_freq[kMaxRopePairs];   // base^(-2i/d_r), computed once on the host in fp64
};

// fp64 -> bf16, round to nearest even without double rounding: truncate to f32 toward zero, fold
// everything that was cut off into the f32's last mantissa bit (round to odd), then round that
// f32 to 8 significant bits.  f32 keeps 16 more bits than bf16, so the two-step result equals the
// direct rounding of the fp64 value.
__device__ __forceinline__ uint16_t double_to_bf16_bits(double x) {
    float f = __double2float_rz(x);
    uint32_t u = __float_as_uint(f);
    if ((double)f != x && (u & 0x7f800000u) != 0x7f800000u) u |= 1u;
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);   // NaN stays NaN
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
// 8-bit e4m3 codes: round to nearest even, finite overflow and infinity saturate to +-448, NaN stays NaN
__device__ __forceinline__ uint8_t float_to_e4m3_bits(float f) { return (uint8_t)__nv_cvt_float_to_fp8(f, __NV_SATFINITE, __NV_E4M3); }
__device__ __forceinline__ uint8_t double_to_e4m3_bits(double x) { return (uint8_t)__nv_cvt_double_to_fp8(x, __NV_SATFINITE, __NV_E4M3); }

// One pair of y = x R_pos^T in fp64.
__device__ __forceinline__ void rope_pair(double x0, double x1, int pos, double inv_freq, double &y0, double &y1) {
    double s, c;
    sincos((double)pos * inv_freq, &s, &c);
    y0 = x0 * c - x1 * s;
    y1 = x0 * s + x1 * c;
}

// ---- absorb --------------------------------------------------------------------------------------
// grid (H, ceil(B / kAbsorbBatch)), block 256.  M_h is staged once per block in shared memory
// (row stride d_c + 4 floats: 16-byte aligned for cp.async and conflict-free for 16-byte row-per-thread
// reads), and reused for kAbsorbBatch sequences.
constexpr int kAbsorbBatch = 8;
constexpr int kAbsorbBatchMax = 16;      // the fused front of a decode step takes 16 sequences per block for large batches of
                                         // the 64-wide shape, so that its grid stays at one block per SM (see step_front_kernel)
constexpr int kAbsorbThreads = 256;

// Shared-memory row stride of the staged map, in floats: d_c + 4 keeps rows 16-byte aligned for cp.async.
__host__ __device__ __forceinline__ int absorb_row_stride(int d_c) { return d_c + 4; }
__host__ __device__ __forceinline__ size_t absorb_smem_bytes(int d_v, int d_c) {
    return ((size_t)d_v * absorb_row_stride(d_c) + (size_t)kAbsorbBatchMax * d_c) * sizeof(float);
}

// One block's share: head h, sequences [b0, b0 + batch), batch <= kAbsorbBatchMax.  All kAbsorbThreads threads must call it.
// Every global read is requested up front -- M_h and the query rows as 16-byte cp.async copies straight into
// shared memory, the RoPE inputs into registers -- so the block pays one memory round trip.
// `overlap` is called once by every thread while the copies are in flight (a caller's own latency-bound work).
struct NoOverlap {
    __device__ __forceinline__ void operator()() const {}
};
// Requests M_h into the block's shared memory ahead of absorb_block (which is then told that the map is in flight).
// Returns false when the pointers do not allow 16-byte copies: absorb_block then loads the map itself.
__device__ __forceinline__ bool absorb_prefetch_map(const float *__restrict__ q_c, const float *__restrict__ M, int d_v, int d_c,
                                                    int h, float *smem_f) {
    const bool vec = (d_c & 3) == 0 && (reinterpret_cast<uintptr_t>(q_c) & 15) == 0 && (reinterpret_cast<uintptr_t>(M) & 15) == 0;
    if (!vec) return false;
    const int ld = absorb_row_stride(d_c), cpr = d_c >> 2;
    const float *Mh = M + (size_t)h * d_v * d_c;
    const uint32_t sM_u32 = smem_u32(smem_f);
    for (int c = threadIdx.x; c < d_v * cpr; c += kAbsorbThreads) {
        const int row = c / cpr, col = c % cpr;
        cp_async16(sM_u32 + (row * ld + col * 4) * 4, Mh + (size_t)row * d_c + col * 4, 16);
    }
    cp_async_commit();
    return true;
}
template <typename Overlap = NoOverlap>
__device__ __forceinline__ void absorb_block(const float *__restrict__ q_c, const float *__restrict__ q_r,
                                             const float *__restrict__ M, const int32_t *__restrict__ q_pos,
                                             float *__restrict__ q_abs, int B, int H, int d_v, int d_c, int d_r,
                                             const RopeTable &rope, int h, int b0, float *smem_f, int batch = kAbsorbBatch,
                                             Overlap overlap = Overlap(), bool map_in_flight = false) {
    const int ld = absorb_row_stride(d_c);
    float *sM = smem_f;                            // [d_v][ld]
    float *sq = smem_f + d_v * ld;                 // [batch][d_c]
    const int nb = min(batch, B - b0);
    const int tid = threadIdx.x;
    const float *Mh = M + (size_t)h * d_v * d_c;
    const int dq = d_v + d_r;
    const int half = d_r / 2;
    const bool vec = (d_c & 3) == 0 && (reinterpret_cast<uintptr_t>(q_c) & 15) == 0 && (reinterpret_cast<uintptr_t>(M) & 15) == 0;
    if (vec) {
        const int cpr = d_c >> 2;                  // 16-byte chunks per row
        const uint32_t sM_u32 = smem_u32(sM), sq_u32 = smem_u32(sq);
        if (!map_in_flight) {
            for (int c = tid; c < d_v * cpr; c += kAbsorbThreads) {
                const int row = c / cpr, col = c % cpr;
                cp_async16(sM_u32 + (row * ld + col * 4) * 4, Mh + (size_t)row * d_c + col * 4, 16);
            }
        }
        for (int c = tid; c < nb * cpr; c += kAbsorbThreads) {
            const int bb = c / cpr, col = c % cpr;
            cp_async16(sq_u32 + (bb * d_c + col * 4) * 4, q_c + ((size_t)(b0 + bb) * H + h) * d_c + col * 4, 16);
        }
        cp_async_commit();
    } else {
        for (int i = tid; i < d_v * d_c; i += kAbsorbThreads) sM[(i / d_c) * ld + (i % d_c)] = Mh[i];
        for (int i = tid; i < nb * d_c; i += kAbsorbThreads)
            sq[i] = q_c[((size_t)(b0 + i / d_c) * H + h) * d_c + (i % d_c)];
    }
    float r0 = 0.f, r1 = 0.f;
    int rpos = 0;
    const bool has_rope = tid < nb * half;      // nb * half <= 16 * 16 = kAbsorbThreads
    if (has_rope) {
        const int bb = tid / half, i = tid % half;
        const size_t src = ((size_t)(b0 + bb) * H + h) * d_r + 2 * i;
        r0 = q_r[src];
        r1 = q_r[src + 1];
        rpos = q_pos[b0 + bb];
    }
    if (has_rope) {                             // the rotation overlaps with the copies in flight
        const int bb = tid / half, i = tid % half;
        double y0, y1;
        rope_pair((double)r0, (double)r1, rpos, rope.inv_freq[i], y0, y1);
        float *dst = q_abs + ((size_t)(b0 + bb) * H + h) * dq + d_v + 2 * i;
        dst[0] = __double2float_rn(y0);
        dst[1] = __double2float_rn(y1);
    }
    overlap();
    if (vec) cp_async_wait<0>();
    __syncthreads();
    // Thread t owns map row i = t % d_v for sequences bb0, bb0 + step, ... (kAbsorbThreads % d_v == 0), so one
    // read of M_h[i][j] feeds up to four independent accumulators.
    if (kAbsorbThreads % d_v == 0 && batch * d_v <= 4 * kAbsorbThreads) {
        const int i = tid % d_v, bb0 = tid / d_v, step = kAbsorbThreads / d_v;
        const float *mrow = sM + i * ld;
        const float *q0 = sq + min(bb0, nb - 1) * d_c, *q1 = sq + min(bb0 + step, nb - 1) * d_c;
        const float *q2 = sq + min(bb0 + 2 * step, nb - 1) * d_c, *q3 = sq + min(bb0 + 3 * step, nb - 1) * d_c;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        if (vec) {      // 16-byte shared-memory reads: rows are 16-byte aligned and (d_c + 4) * 4 bytes apart, conflict-free
            const float4 *m4 = reinterpret_cast<const float4 *>(mrow);
            const float4 *p0 = reinterpret_cast<const float4 *>(q0), *p1 = reinterpret_cast<const float4 *>(q1);
            const float4 *p2 = reinterpret_cast<const float4 *>(q2), *p3 = reinterpret_cast<const float4 *>(q3);
#pragma unroll 2
            for (int j = 0; j < (d_c >> 2); ++j) {
                const float4 m = m4[j], x0 = p0[j], x1 = p1[j], x2 = p2[j], x3 = p3[j];
                a0 = fmaf(x0.x, m.x, a0); a0 = fmaf(x0.y, m.y, a0); a0 = fmaf(x0.z, m.z, a0); a0 = fmaf(x0.w, m.w, a0);
                a1 = fmaf(x1.x, m.x, a1); a1 = fmaf(x1.y, m.y, a1); a1 = fmaf(x1.z, m.z, a1); a1 = fmaf(x1.w, m.w, a1);
                a2 = fmaf(x2.x, m.x, a2); a2 = fmaf(x2.y, m.y, a2); a2 = fmaf(x2.z, m.z, a2); a2 = fmaf(x2.w, m.w, a2);
                a3 = fmaf(x3.x, m.x, a3); a3 = fmaf(x3.y, m.y, a3); a3 = fmaf(x3.z, m.z, a3); a3 = fmaf(x3.w, m.w, a3);
            }
        } else {
#pragma unroll 4
            for (int j = 0; j < d_c; ++j) {
                const float m = mrow[j];
                a0 = fmaf(q0[j], m, a0);
                a1 = fmaf(q1[j], m, a1);
                a2 = fmaf(q2[j], m, a2);
                a3 = fmaf(q3[j], m, a3);
            }
        }
        const float acc[4] = {a0, a1, a2, a3};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int bb = bb0 + k * step;
            if (bb < nb) q_abs[((size_t)(b0 + bb) * H + h) * dq + i] = acc[k];
        }
    } else {
        for (int o = tid; o < nb * d_v; o += kAbsorbThreads) {
            const int bb = o / d_v, i = o % d_v;
            const float *mrow = sM + i * ld;
            const float *qrow = sq + bb * d_c;
            float acc = 0.f;
            for (int j = 0; j < d_c; ++j) acc = fmaf(qrow[j], mrow[j], acc);
            q_abs[((size_t)(b0 + bb) * H + h) * dq + i] = acc;
        }
    }
}

__global__ void __launch_bounds__(kAbsorbThreads)
absorb_kernel(const float *__restrict__ q_c, const float *__restrict__ q_r, const float *__restrict__ M,
              const int32_t *__restrict__ q_pos, float *__restrict__ q_abs, int B, int H, int d_v, int d_c,
              int d_r, RopeTable rope) {
    grid_dependency_launch();
    extern __shared__ float smem_f[];
    const bool map_in_flight = absorb_prefetch_map(q_c, M, d_v, d_c, blockIdx.x, smem_f);      // (a weight: see step_front_kernel)
    grid_dependency_wait();
    absorb_block(q_c, q_r, M, q_pos, q_abs, B, H, d_v, d_c, d_r, rope, blockIdx.x, blockIdx.y * kAbsorbBatch, smem_f, kAbsorbBatch,
                 NoOverlap(), map_in_flight);
}

// ---- absorb for many rows on the tensor cores --------------------------------------------------------
// The same product as a batch of small GEMMs, Q_abs[:, h, :d_v] = Q_c[:, h, :] M_h^T, with f32-level accuracy from f16
// MMAs: both operands are split x = hi + lo (f16 each, 22 significant bits together) and hi*hi + hi*lo + lo*hi is
// accumulated in f32 (the dropped lo*lo term is below 2^-22 relative).  grid (H, blocks per head), block 128: M_h's two
// halves sit in shared memory as f16 [d_v][d_c] (rows padded by 8 so that the ldmatrix fetches of B fragments are conflict-free); each warp
// walks its own 16-row tiles of the block's strip, fetching the A fragments straight from global memory (a warp-wide
// load covers whole 32-byte sectors) one tile ahead, so that no barrier and no staging buffer sits on the stream.
// The rotated positional slice is computed as in the other absorb kernels (fp64, one rounding), but once per row for all
// heads: the H blocks that share a strip of rows split its rows among themselves.
__device__ __forceinline__ void mma_m16n8k16_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split_f16x2(float x, float y, uint32_t &hi, uint32_t &lo) {
    const __half2 h = __floats2half2_rn(x, y);
    const float2 f = __half22float2(h);
    const __half2 l = __floats2half2_rn(x - f.x, y - f.y);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = *reinterpret_cast<const uint32_t *>(&l);
}
__device__ __forceinline__ void absorb_ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
constexpr int kAbsorbMmaThreads = 128;
constexpr int kAbsorbMmaRows = (kAbsorbMmaThreads / 32) * 16;       // rows a block covers per round of its warps
template <int DV, int DC>
struct AbsorbMmaTraits {
    static constexpr int MLD = DC + 8;                              // f16 elements per row of a map half
    static constexpr size_t smem_bytes() { return (size_t)2 * DV * MLD * 2; }
};
template <int DV, int DC>
__global__ void __launch_bounds__(kAbsorbMmaThreads, DV == 64 ? 4 : 2)
absorb_rows_mma_kernel(const float *__restrict__ q_c, const float *__restrict__ q_r, const float *__restrict__ M,
                       const int32_t *__restrict__ q_pos, float *__restrict__ q_abs, int B, int H, int d_r, int rows_per_block,
                       RopeTable rope) {
    using T = AbsorbMmaTraits<DV, DC>;
    constexpr int MLD = T::MLD, NT = DV / 8, KS = DC / 16;
    grid_dependency_launch();
    extern __shared__ __align__(16) unsigned char absorb_smem[];
    __half *m_hi = reinterpret_cast<__half *>(absorb_smem);
    __half *m_lo = m_hi + DV * MLD;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, h = blockIdx.x;
    const int g = lane >> 2, t = lane & 3;
    const int row0 = blockIdx.y * rows_per_block;
    const int row1 = min(B, row0 + rows_per_block);
    grid_dependency_wait();
    if (row0 >= row1) return;
    // the map, split once per block
    for (int e = tid; e < DV * DC / 2; e += kAbsorbMmaThreads) {
        const int i = e / (DC / 2), j = (e % (DC / 2)) * 2;
        const float2 v = *reinterpret_cast<const float2 *>(M + ((size_t)h * DV + i) * DC + j);
        uint32_t hi, lo;
        split_f16x2(v.x, v.y, hi, lo);
        *reinterpret_cast<uint32_t *>(m_hi + i * MLD + j) = hi;
        *reinterpret_cast<uint32_t *>(m_lo + i * MLD + j) = lo;
    }
    const int dq = DV + d_r, half = d_r / 2;
    // the positional slices of this block's share of the strip: one (row, pair) per thread and pass, all heads
    {
        const int n = row1 - row0, per = (n + H - 1) / H, lo = min(n, h * per), cnt = min(n, lo + per) - lo;
        for (int e = tid; e < cnt * half; e += kAbsorbMmaThreads) {
            const int row = row0 + lo + e / half, k = e % half;
            double sn, cs;
            sincos((double)q_pos[row] * rope.inv_freq[k], &sn, &cs);
            const float *src = q_r + (size_t)row * H * d_r + 2 * k;
            float *dst = q_abs + (size_t)row * H * dq + DV + 2 * k;
            for (int h0 = 0; h0 < H; h0 += 8) {
                float2 x[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)      // eight independent loads in flight
                    x[u] = (h0 + u < H) ? *reinterpret_cast<const float2 *>(src + (size_t)(h0 + u) * d_r) : make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const double x0 = (double)x[u].x, x1 = (double)x[u].y;
                    if (h0 + u < H)
                        *reinterpret_cast<float2 *>(dst + (size_t)(h0 + u) * dq) =
                            make_float2(__double2float_rn(x0 * cs - x1 * sn), __double2float_rn(x0 * sn + x1 * cs));
                }
            }
        }
    }
    __syncthreads();                // the split map is visible to every warp
    // A fragments of one 16-row tile: rows g and g + 8, k = 16 ks + 2t, +1 and + 8, + 9 -- 8 bytes per lane and load
    auto fetch = [&](int r0, float2 (&x)[KS][4]) {
        const int ra = min(r0 + g, row1 - 1), rb = min(r0 + g + 8, row1 - 1);      // rows past the end repeat the last one
        const float *pa = q_c + ((size_t)ra * H + h) * DC + 2 * t;
        const float *pb = q_c + ((size_t)rb * H + h) * DC + 2 * t;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            x[ks][0] = *reinterpret_cast<const float2 *>(pa + ks * 16);
            x[ks][1] = *reinterpret_cast<const float2 *>(pb + ks * 16);
            x[ks][2] = *reinterpret_cast<const float2 *>(pa + ks * 16 + 8);
            x[ks][3] = *reinterpret_cast<const float2 *>(pb + ks * 16 + 8);
        }
    };
    // ldmatrix row address of this lane: matrices (n-tile, k 0-7), (n-tile, k 8-15), (n-tile + 1, k 0-7), (n-tile + 1, k 8-15)
    const int b_off = (((lane >> 4) * 8 + (lane & 7)) * MLD + ((lane >> 3) & 1) * 8) * 2;
    const uint32_t b_hi_addr = smem_u32(m_hi) + b_off, b_lo_addr = smem_u32(m_lo) + b_off;
    float2 cur[KS][4], nxt[KS][4];
    int r0 = row0 + warp * 16;
    if (r0 < row1) fetch(r0, cur);
    for (; r0 < row1; r0 += kAbsorbMmaRows) {
        const int rn = r0 + kAbsorbMmaRows;
        if (rn < row1) fetch(rn, nxt);
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t a_hi[4], a_lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) split_f16x2(cur[ks][e].x, cur[ks][e].y, a_hi[e], a_lo[e]);
#pragma unroll
            for (int nt = 0; nt < NT; nt += 2) {
                // B = M_h^T: element (k, n) is M_h[n][k]; a fragment register is two consecutive k of one n, which is what
                // ldmatrix hands out from the [n][k] rows: one fetch = (k 0-7 | k 8-15) of n-tiles nt and nt + 1
                uint32_t bh[4], bl[4];
                absorb_ldsm_x4(b_hi_addr + (nt * 8 * MLD + ks * 16) * 2, bh);
                absorb_ldsm_x4(b_lo_addr + (nt * 8 * MLD + ks * 16) * 2, bl);
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    mma_m16n8k16_f16(acc[nt + u], a_lo, bh[2 * u], bh[2 * u + 1]);      // small terms first
                    mma_m16n8k16_f16(acc[nt + u], a_hi, bl[2 * u], bl[2 * u + 1]);
                    mma_m16n8k16_f16(acc[nt + u], a_hi, bh[2 * u], bh[2 * u + 1]);
                }
            }
        }
        const int ra = r0 + g, rb = ra + 8;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            if (ra < row1)
                *reinterpret_cast<float2 *>(q_abs + ((size_t)ra * H + h) * dq + nt * 8 + 2 * t) = make_float2(acc[nt][0], acc[nt][1]);
            if (rb < row1)
                *reinterpret_cast<float2 *>(q_abs + ((size_t)rb * H + h) * dq + nt * 8 + 2 * t) = make_float2(acc[nt][2], acc[nt][3]);
        }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int e = 0; e < 4; ++e) cur[ks][e] = nxt[ks][e];
    }
}

// ---- append --------------------------------------------------------------------------------------
// grid B, block 128.  Integer page arithmetic, round-to-nearest-even stores, nothing else touched.
// The new rows are loaded before the page lookup so that the two dependent lookups (position, then
// block-table entry) overlap with them.
constexpr int kAppendMaxPerThread = 8;    // G * d_v <= 8 * 128 elements (blocks have at least 128 threads)

// One sequence's append in steps, so that a caller can put other work between the loads and what depends on them:
// append_load requests the new row (nothing it returns is looked at yet), append_locate looks up the page of position t
// (a dependent load: the position itself usually comes from memory), append_rotate rotates the positional pair,
// append_store checks the page, rounds and writes.  Every thread of the block must call all four (blockDim.x >= 128).
// Input row `row` (v_new[row], kr_new[row]) becomes token `t` of sequence `seq`.
struct AppendRegs {
    float x[kAppendMaxPerThread];
    float k0, k1;
    double y0, y1;       // the rotated pair, once append_rotate has run
    long long page;      // as looked up; checked by append_store
    int t;               // -1: position outside the block table (reported by append_locate), nothing is written
    int rope_tid0;       // threads [rope_tid0, rope_tid0 + d_r / 2) hold the positional pairs
};
__device__ __forceinline__ AppendRegs append_load(const float *__restrict__ v_new, const float *__restrict__ kr_new, int G,
                                                  int d_v, int d_r, int row, int rope_tid0 = 0) {
    AppendRegs r;
    r.rope_tid0 = rope_tid0;
    const int n_v = G * d_v;
    const int nt = blockDim.x;
#pragma unroll
    for (int u = 0; u < kAppendMaxPerThread; ++u) {
        const int i = u * nt + threadIdx.x;
        r.x[u] = (i < n_v) ? v_new[(size_t)row * n_v + i] : 0.f;
    }
    r.k0 = r.k1 = 0.f;
    const int rk = (int)threadIdx.x - rope_tid0;
    if (rk >= 0 && rk < d_r / 2) {
        r.k0 = kr_new[(size_t)row * d_r + 2 * rk];
        r.k1 = kr_new[(size_t)row * d_r + 2 * rk + 1];
    }
    r.t = -1;
    r.page = -1;
    r.y0 = r.y1 = 0.0;
    return r;
}
__device__ __forceinline__ void append_locate(AppendRegs &r, const int32_t *__restrict__ block_table, int P, int max_pages,
                                              int32_t *dev_status, int seq, int t) {
    if (t < 0 || t / P >= max_pages) {
        if (threadIdx.x == 0) report_error(dev_status, GVA_ERR_SEQ_LEN, seq);
        return;
    }
    r.t = t;
    r.page = block_table ? (long long)block_table[(size_t)seq * max_pages + t / P] : (long long)seq * max_pages + t / P;
}
// The rotation of the positional pair (fp64).
__device__ __forceinline__ void append_rotate(AppendRegs &r, int d_r, const RopeTable &rope) {
    const int i = (int)threadIdx.x - r.rope_tid0;
    if (r.t >= 0 && i >= 0 && i < d_r / 2) rope_pair((double)r.k0, (double)r.k1, r.t, rope.inv_freq[i], r.y0, r.y1);
}
template <typename CT>
__device__ __forceinline__ void append_store(const AppendRegs &r, CT *__restrict__ v_pool, CT *__restrict__ kr_pool, int G,
                                             int d_v, int d_r, int P, int num_pages, int32_t *dev_status, int seq) {
    if (r.t < 0) return;
    if (r.page < 0 || r.page >= num_pages) {
        if (threadIdx.x == 0) report_error(dev_status, GVA_ERR_BAD_PAGE, seq);
        return;
    }
    const int n_v = G * d_v;
    const int nt = blockDim.x;
    const long long page = r.page;
    const int slot = r.t % P;
#pragma unroll
    for (int u = 0; u < kAppendMaxPerThread; ++u) {
        const int i = u * nt + threadIdx.x;
        if (i < n_v) {
            const int g = i / d_v, d = i % d_v;
            const size_t dst = (((size_t)page * G + g) * P + slot) * d_v + d;
            if constexpr (sizeof(CT) == 1) reinterpret_cast<uint8_t *>(v_pool)[dst] = float_to_e4m3_bits(r.x[u]);
            else if constexpr (sizeof(CT) == 2) reinterpret_cast<uint16_t *>(v_pool)[dst] = float_to_bf16_bits(r.x[u]);
            else reinterpret_cast<float *>(v_pool)[dst] = r.x[u];
        }
    }
    const int i = (int)threadIdx.x - r.rope_tid0;
    if (i >= 0 && i < d_r / 2) {
        const double y0 = r.y0, y1 = r.y1;
        const size_t dst = ((size_t)page * P + slot) * d_r + 2 * i;
        if constexpr (sizeof(CT) == 1) {
            reinterpret_cast<uint8_t *>(kr_pool)[dst] = double_to_e4m3_bits(y0);
            reinterpret_cast<uint8_t *>(kr_pool)[dst + 1] = double_to_e4m3_bits(y1);
        } else if constexpr (sizeof(CT) == 2) {
            reinterpret_cast<uint16_t *>(kr_pool)[dst] = double_to_bf16_bits(y0);
            reinterpret_cast<uint16_t *>(kr_pool)[dst + 1] = double_to_bf16_bits(y1);
        } else {
            reinterpret_cast<float *>(kr_pool)[dst] = __double2float_rn(y0);
            reinterpret_cast<float *>(kr_pool)[dst + 1] = __double2float_rn(y1);
        }
    }
}
template <typename CT>
__device__ __forceinline__ void append_row(CT *__restrict__ v_pool, CT *__restrict__ kr_pool,
                                           const int32_t *__restrict__ block_table, const float *__restrict__ v_new,
                                           const float *__restrict__ kr_new, int G, int d_v, int d_r, int P, int num_pages,
                                           int max_pages, int32_t *dev_status, const RopeTable &rope, int row, int seq, int t) {
    AppendRegs r = append_load(v_new, kr_new, G, d_v, d_r, row);
    append_locate(r, block_table, P, max_pages, dev_status, seq, t);
    append_rotate(r, d_r, rope);
    append_store<CT>(r, v_pool, kr_pool, G, d_v, d_r, P, num_pages, dev_status, seq);
}

template <typename CT>
__device__ __forceinline__ void append_block(CT *__restrict__ v_pool, CT *__restrict__ kr_pool,
                                             const int32_t *__restrict__ block_table, const float *__restrict__ v_new,
                                             const float *__restrict__ kr_new, const int32_t *__restrict__ pos, int G,
                                             int d_v, int d_r, int P, int num_pages, int max_pages, int32_t *dev_status,
                                             const RopeTable &rope, int b) {
    append_row<CT>(v_pool, kr_pool, block_table, v_new, kr_new, G, d_v, d_r, P, num_pages, max_pages, dev_status, rope, b, b,
                   pos[b]);
}

template <typename CT>
__global__ void __launch_bounds__(128)
append_kernel(CT *__restrict__ v_pool, CT *__restrict__ kr_pool, const int32_t *__restrict__ block_table,
              const float *__restrict__ v_new, const float *__restrict__ kr_new, const int32_t *__restrict__ pos,
              int G, int d_v, int d_r, int P, int num_pages, int max_pages, int32_t *dev_status, RopeTable rope) {
    grid_dependency_launch();
    grid_dependency_wait();
    append_block<CT>(v_pool, kr_pool, block_table, v_new, kr_new, pos, G, d_v, d_r, P, num_pages, max_pages, dev_status,
                     rope, blockIdx.x);
}

// Append of a chunk of new tokens per sequence: input row n becomes token ctx_lens[b] + (n - cu_q[b]) of the sequence b
// that owns the row (found by bisection of cu_q).  A block writes kAppendChunkRows consecutive rows, all at once: 16
// threads per row first resolve the row's page and slot and write its rotated positional key (one pair each, fp64), then
// the whole block copies the value rows with every load independent of the others.
constexpr int kAppendChunkRows = 8;
template <typename CT>
__global__ void __launch_bounds__(128)
append_chunk_kernel(CT *__restrict__ v_pool, CT *__restrict__ kr_pool, const int32_t *__restrict__ block_table,
                    const float *__restrict__ v_new, const float *__restrict__ kr_new, const int32_t *__restrict__ cu_q,
                    const int32_t *__restrict__ ctx_lens, int B, int G, int d_v, int d_r, int P, int num_pages, int max_pages,
                    int32_t *dev_status, RopeTable rope, int vec4) {
    static_assert(kAppendChunkRows * kMaxRopePairs == 128, "16 threads per row");
    grid_dependency_launch();
    __shared__ long long s_page[kAppendChunkRows];      // -1: the row is not written
    __shared__ int s_slot[kAppendChunkRows];
    grid_dependency_wait();
    const int total = cu_q[B];
    {
        const int r = threadIdx.x / kMaxRopePairs, k = threadIdx.x % kMaxRopePairs;
        const int n = blockIdx.x * kAppendChunkRows + r;
        long long page = -1;
        int slot = 0;
        if (n < total) {
            int lo = 0, hi = B - 1;                     // largest b with cu_q[b] <= n (empty sequences repeat an offset)
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (cu_q[mid] <= n) lo = mid;
                else hi = mid - 1;
            }
            const int b = lo, t = ctx_lens[b] + (n - cu_q[b]);
            float k0 = 0.f, k1 = 0.f;
            if (k < d_r / 2) {
                k0 = kr_new[(size_t)n * d_r + 2 * k];
                k1 = kr_new[(size_t)n * d_r + 2 * k + 1];
            }
            if (t < 0 || t / P >= max_pages) {
                if (k == 0) report_error(dev_status, GVA_ERR_SEQ_LEN, b);
            } else {
                page = block_table ? (long long)block_table[(size_t)b * max_pages + t / P] : (long long)b * max_pages + t / P;
                slot = t % P;
                if (page < 0 || page >= num_pages) {
                    if (k == 0) report_error(dev_status, GVA_ERR_BAD_PAGE, b);
                    page = -1;
                } else if (k < d_r / 2) {
                    double y0, y1;
                    rope_pair((double)k0, (double)k1, t, rope.inv_freq[k], y0, y1);
                    const size_t dst = ((size_t)page * P + slot) * d_r + 2 * k;
                    if constexpr (sizeof(CT) == 1) {
                        reinterpret_cast<uint8_t *>(kr_pool)[dst] = double_to_e4m3_bits(y0);
                        reinterpret_cast<uint8_t *>(kr_pool)[dst + 1] = double_to_e4m3_bits(y1);
                    } else if constexpr (sizeof(CT) == 2) {
                        reinterpret_cast<uint16_t *>(kr_pool)[dst] = double_to_bf16_bits(y0);
                        reinterpret_cast<uint16_t *>(kr_pool)[dst + 1] = double_to_bf16_bits(y1);
                    } else {
                        reinterpret_cast<float *>(kr_pool)[dst] = __double2float_rn(y0);
                        reinterpret_cast<float *>(kr_pool)[dst + 1] = __double2float_rn(y1);
                    }
                }
            }
        }
        if (k == 0) {
            s_page[r] = page;
            s_slot[r] = slot;
        }
    }
    __syncthreads();
    const int n_v = G * d_v;
    const int rows = min(kAppendChunkRows, total - (int)blockIdx.x * kAppendChunkRows);
    const float *src = v_new + (size_t)blockIdx.x * kAppendChunkRows * n_v;
    // element e = r * n_v + i walks the rows in steps of 128 without a division (d_v is a power of two: 64 or 128)
    const int sh = 31 - __clz(d_v);
    if (vec4) {     // v_new is 16-byte aligned: four elements per thread and pass
        const int n4 = n_v >> 2;
        int r = 0, i = threadIdx.x;
        while (i >= n4) {
            i -= n4;
            ++r;
        }
        while (r < rows) {
            const long long page = s_page[r];
            if (page >= 0) {
                const int g = (4 * i) >> sh, d = (4 * i) & (d_v - 1);
                const size_t dst = (((size_t)page * G + g) * P + s_slot[r]) * d_v + d;
                const float4 x = *reinterpret_cast<const float4 *>(src + (size_t)r * n_v + 4 * i);
                if constexpr (sizeof(CT) == 1) {
                    *reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(v_pool) + dst) =
                        (uint32_t)float_to_e4m3_bits(x.x) | ((uint32_t)float_to_e4m3_bits(x.y) << 8) |
                        ((uint32_t)float_to_e4m3_bits(x.z) << 16) | ((uint32_t)float_to_e4m3_bits(x.w) << 24);
                } else if constexpr (sizeof(CT) == 2) {
                    *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(v_pool) + dst) =
                        make_uint2((uint32_t)float_to_bf16_bits(x.x) | ((uint32_t)float_to_bf16_bits(x.y) << 16),
                                   (uint32_t)float_to_bf16_bits(x.z) | ((uint32_t)float_to_bf16_bits(x.w) << 16));
                } else {
                    *reinterpret_cast<float4 *>(reinterpret_cast<float *>(v_pool) + dst) = x;
                }
            }
            i += 128;
            while (i >= n4) {
                i -= n4;
                ++r;
            }
        }
        return;
    }
    int r = 0, i = threadIdx.x;
    while (i >= n_v) {
        i -= n_v;
        ++r;
    }
    while (r < rows) {
        const long long page = s_page[r];
        if (page >= 0) {
            const int g = i >> sh, d = i & (d_v - 1);
            const size_t dst = (((size_t)page * G + g) * P + s_slot[r]) * d_v + d;
            const float x = src[(size_t)r * n_v + i];
            if constexpr (sizeof(CT) == 1) reinterpret_cast<uint8_t *>(v_pool)[dst] = float_to_e4m3_bits(x);
            else if constexpr (sizeof(CT) == 2) reinterpret_cast<uint16_t *>(v_pool)[dst] = float_to_bf16_bits(x);
            else reinterpret_cast<float *>(v_pool)[dst] = x;
        }
        i += 128;
        while (i >= n_v) {
            i -= n_v;
            ++r;
        }
    }
}

// Brings two small int32 arrays that live in pinned host memory into device scratch: one block reading them over the
// interconnect costs less stream time than two copy-engine transfers.
__global__ void __launch_bounds__(128)
stage_ints_kernel(const int32_t *__restrict__ a_src, const int32_t *__restrict__ b_src, int32_t *__restrict__ a_dst,
                  int32_t *__restrict__ b_dst, int n) {
    grid_dependency_launch();
    grid_dependency_wait();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int32_t x = a_src[i], y = b_src[i];
        a_dst[i] = x;
        b_dst[i] = y;
    }
}

// ---- fused front of a decode step: absorb and append in one launch ------------------------------------
// Absorb items (head = item % H, batch tile = item / H) and one append per sequence, independent of each other; which
// block runs what is described in the kernel.  This kernel
// waits for everything earlier in the stream BEFORE it lets its dependent (the decode kernel) start, so
// whatever the decode kernel does ahead of its own wait overlaps with this kernel only.
struct StepFrontParams {
    const float *q_c, *q_r, *M, *v_new, *kr_new;
    const int32_t *pos, *block_table;
    float *q_abs;
    void *v_pool, *kr_pool;
    int32_t *dev_status;
    int B, H, G, d_v, d_c, d_r, P, num_pages, max_pages, n_absorb;
    int trace_call;      // number of the decode call this launch belongs to (timeline builds only)
    int batch;           // sequences per absorb item: kAbsorbBatch or kAbsorbBatchMax
    int fold;            // 1: the first B blocks append as well (grid = max(n_absorb, B)); 0: appends have blocks of their own
};

template <typename CT>
__global__ void __launch_bounds__(kAbsorbThreads)
step_front_kernel(StepFrontParams a, RopeTable rope) {
    extern __shared__ float smem_f[];
    // The map M_h is a weight: it is requested before the wait for the preceding work in the stream (in a decode loop the
    // merge kernel of the previous step), so that its round trip is over when the step's own inputs may be read.
    bool map_in_flight = false;
    if ((int)blockIdx.x < a.n_absorb) map_in_flight = absorb_prefetch_map(a.q_c, a.M, a.d_v, a.d_c, blockIdx.x % a.H, smem_f);
    grid_dependency_wait();
    grid_dependency_launch();
    if (threadIdx.x == 0) trace(kTrFrontEnterMin, a.trace_call);
    // Small batches: blocks [0, n_absorb) run one absorb item each, blocks [n_absorb, n_absorb + B) one append each.
    // Batches whose grid would exceed one block per SM (fold): block x runs absorb item x (x < n_absorb) AND appends sequence
    // x's new token (x < B), and the 64-wide shape takes 16 sequences per absorb item -- the blocks of this kernel share
    // their SMs with the decode blocks that were started early, which leave room for one of them at a time, so every block
    // beyond one per SM is another round.  A folded append requests its loads first, so that they share the absorb item's
    // memory round trip; its dependent page lookup and its rotation run while the item's copies fly.
    const int seq_app = a.fold ? (int)blockIdx.x : (int)blockIdx.x - a.n_absorb;
    const bool appends = seq_app >= 0 && seq_app < a.B;
    AppendRegs ar;
    int t_app = 0;
    if (appends) {     // (its positional pairs sit in the last warp: the first ones rotate the query's)
        t_app = a.pos[seq_app];
        ar = append_load(a.v_new, a.kr_new, a.G, a.d_v, a.d_r, seq_app, kAbsorbThreads - 32);
    }
    auto locate_and_rotate = [&]() {
        if (appends) {
            append_locate(ar, a.block_table, a.P, a.max_pages, a.dev_status, seq_app, t_app);
            append_rotate(ar, a.d_r, rope);
        }
    };
    if ((int)blockIdx.x < a.n_absorb) {
        absorb_block(a.q_c, a.q_r, a.M, a.pos, a.q_abs, a.B, a.H, a.d_v, a.d_c, a.d_r, rope, blockIdx.x % a.H,
                     (blockIdx.x / a.H) * a.batch, smem_f, a.batch, locate_and_rotate, map_in_flight);
    } else {
        locate_and_rotate();
    }
    if (appends)
        append_store<CT>(ar, static_cast<CT *>(a.v_pool), static_cast<CT *>(a.kr_pool), a.G, a.d_v, a.d_r, a.P, a.num_pages,
                         a.dev_status, seq_app);
    if (threadIdx.x == 0) trace(kTrFrontExitMax, a.trace_call);
}

// ---- LSE combine ---------------------------------------------------------------------------------
// A block holds hpb heads of one sequence, wph warps per head (blockDim = 32 * wph * hpb, grid (B, H / hpb)).
// Warp `part` of a head takes records part, part + wph, ...; eight records' (max, sum) pairs and partial outputs
// are requested before any is used, so a head covers 8 * wph records per memory round trip.  Each warp keeps a
// running (m, L, acc) by the usual rescaling and the wph warp states are merged through shared memory in a fixed
// order, so the result is reproducible for fixed launch geometry.  The host picks wph from the number of
// records a sequence can have (many for a single long sequence, few for a large batch).
//   m* = max_r m_r ;  L = sum_r l_r 2^(m_r - m*) ;  out = sum_r 2^(m_r - m*) o_r / L ;  lse = (m* + log2 L) ln 2
//
// The kernel is launched right behind the decode kernel and its blocks become resident while that kernel streams.
// The body runs twice: a first, "dry" pass over record 0 while the block still waits for the decode kernel (loads
// discarded, nothing written), then the real pass after the wait.  Both passes execute the same instructions, so the
// real pass finds them in the SM's instruction cache instead of fetching them cold at the one moment that counts.
template <int DV>
__global__ void __launch_bounds__(1024)
combine_kernel(DecodeParams p, int wph, int hpb) {
    grid_dependency_launch();
    constexpr int DPL = DV / 32;
    constexpr int UNROLL = 8;
    using VecT = typename std::conditional<DPL == 2, float2, float4>::type;
    extern __shared__ float s_comb[];            // [hpb * wph][DV] partial outputs, then [hpb * wph][2] (m, L)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_warps = wph * hpb;
    float *s_acc = s_comb;
    float *s_ml = s_comb + n_warps * DV;
    const int b = blockIdx.x;
    const int h = blockIdx.y * hpb + warp / wph;
    const int part = warp % wph;
    // multi-token decode with its own count per sequence (cu_q): p.H = q_len * H pseudo-heads, of which sequence b uses the
    // first (its count) * H, and its output rows start at cu_q[b]
    const int h_real = p.H / (p.q_len > 1 ? p.q_len : 1);
    size_t out_row0 = (size_t)b * p.H;
    bool active = h < p.H;
    int hh = active ? h : 0;
    if (threadIdx.x == 0) trace(kTrCombineEnterMin, p.epoch);

    // The run of records of this sequence is in the workspace header, which block 0 of the decode kernel publishes as one
    // of the first things it does, followed by the call's stamp.  A merge block that is resident while the decode kernel
    // streams looks for that stamp now and then (one thread, a few polls microseconds apart) and, once it is there,
    // fetches its entry ahead of time: the real pass then starts with the records, not with one more round trip.
    int2 seg_early = make_int2(0, -1);           // y < 0: not fetched
    if (p.num_splits == 0 && p.hdr_stamp != 0) {      // (no stamp: the call is being captured into a graph, see DecodeParams)
        __shared__ int2 s_seg;
        if (threadIdx.x == 0) {
            int2 sg = make_int2(0, -1);
            for (int it = 0; it < 48; ++it) {
                int v;
                asm volatile("ld.acquire.gpu.global.b32 %0, [%1];\n" : "=r"(v) : "l"(p.hdr + kHdrEpoch) : "memory");
                if (v == p.hdr_stamp) {
                    sg = __ldcg(reinterpret_cast<const int2 *>(p.hdr + kHdrInts) + b);
                    break;
                }
                __nanosleep(it < 10 ? 400 : 4000);      // the header comes early in the decode kernel: look closely at first
            }
            s_seg = sg;
        }
        __syncthreads();
        seg_early = s_seg;
    }
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        const bool dry = pass == 0;
        int first = 0, n = 1;                    // dry: record 0 only (always inside the workspace)
        if (!dry) {
            grid_dependency_wait();
            // the decode grid is complete: its tail tickets go back to zero for whoever uses these words next (a later call
            // of the other parity clears them as well; a replay of this very call from a graph relies on this line)
            if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) p.sync[kSyncTicket + (p.epoch & 1)] = 0;
            if (p.cu_q) {      // (an input of the call, but read like everything else only once the stream's earlier work is complete)
                const int r_lo = p.cu_q[b];
                active = h < min(max(p.cu_q[b + 1] - r_lo, 0), p.q_len) * h_real;
                hh = active ? h : 0;
                out_row0 = (size_t)r_lo * h_real;
            }
            if (p.num_splits > 0) {
                first = b * p.num_splits * p.rec_mult;
                n = p.num_splits * p.rec_mult;
            } else {   // this sequence's run of records, worked out by block 0 of the decode kernel
                const int2 seg = seg_early.y >= 0 ? seg_early : __ldcg(reinterpret_cast<const int2 *>(p.hdr + kHdrInts) + b);
                first = seg.x;
                n = seg.y;
            }
            if (n < 0 || first < 0 || first + n > p.n_rec) n = 0;      // a header that cannot be right (a decode kernel that gave up): read nothing
        }
        float m_w = -INFINITY, L_w = 0.f, acc[DPL];
#pragma unroll
        for (int d = 0; d < DPL; ++d) acc[d] = 0.f;
        for (int r0 = part; r0 < n; r0 += wph * UNROLL) {
            float2 ml[UNROLL];
            VecT v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int r = r0 + wph * u;
                ml[u] = make_float2(-INFINITY, 0.f);
                if (r < n) {
                    const size_t rh = (size_t)(first + r) * p.H + hh;
                    ml[u] = __ldcg(reinterpret_cast<const float2 *>(p.rec_ml + rh * 2));
                    v[u] = __ldcg(reinterpret_cast<const VecT *>(p.rec_o + rh * DV + lane * DPL));
                }
            }
            float m_new = m_w;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) m_new = fmaxf(m_new, ml[u].x);
            if (!(m_new > -INFINITY)) continue;          // nothing live yet (or, dry, garbage)
            const float corr = exp2f(m_w - m_new);       // 0 when m_w = -inf
            L_w *= corr;
#pragma unroll
            for (int d = 0; d < DPL; ++d) acc[d] *= corr;
            m_w = m_new;
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (!(ml[u].x > -INFINITY)) continue;    // empty partition or past the end: its output was never written
                const float w = exp2f(ml[u].x - m_new);
                L_w = fmaf(ml[u].y, w, L_w);
                if constexpr (DPL == 2) {
                    acc[0] = fmaf(w, v[u].x, acc[0]);
                    acc[1] = fmaf(w, v[u].y, acc[1]);
                } else {
                    acc[0] = fmaf(w, v[u].x, acc[0]);
                    acc[1] = fmaf(w, v[u].y, acc[1]);
                    acc[2] = fmaf(w, v[u].z, acc[2]);
                    acc[3] = fmaf(w, v[u].w, acc[3]);
                }
            }
        }
        float mstar = m_w, L = L_w, o[DPL];
#pragma unroll
        for (int d = 0; d < DPL; ++d) o[d] = acc[d];
        if (wph > 1) {                                   // block-uniform
            __syncthreads();                             // the previous pass has finished reading shared memory
#pragma unroll
            for (int d = 0; d < DPL; ++d) s_acc[warp * DV + lane * DPL + d] = acc[d];
            if (lane == 0) {
                s_ml[warp * 2] = m_w;
                s_ml[warp * 2 + 1] = L_w;
            }
            __syncthreads();
            if (part == 0) {
                const int w0 = warp;
                mstar = -INFINITY;
                for (int w = 0; w < wph; ++w) mstar = fmaxf(mstar, s_ml[(w0 + w) * 2]);
                L = 0.f;
#pragma unroll
                for (int d = 0; d < DPL; ++d) o[d] = 0.f;
                for (int w = 0; w < wph; ++w) {
                    const float mw = s_ml[(w0 + w) * 2];
                    if (!(mw > -INFINITY)) continue;
                    const float sc = exp2f(mw - mstar);
                    L = fmaf(s_ml[(w0 + w) * 2 + 1], sc, L);
#pragma unroll
                    for (int d = 0; d < DPL; ++d) o[d] = fmaf(sc, s_acc[(w0 + w) * DV + lane * DPL + d], o[d]);
                }
            }
        }
        const bool live = mstar > -INFINITY;
        const float inv = live ? 1.f / L : 0.f;
        const float lse = live ? (mstar + log2f(L)) * kLn2 : -INFINITY;
        if (!dry && active && part == 0) {
            float *o_dst = p.out + (out_row0 + h) * DV + lane * DPL;
#pragma unroll
            for (int d = 0; d < DPL; ++d) o_dst[d] = live ? o[d] * inv : 0.f;
            if (p.lse && lane == 0) p.lse[out_row0 + h] = lse;
            if (lane == 0) {
                trace(kTrCombineOutMin, p.epoch);
                trace(kTrCombineOutMax, p.epoch);
            }
        }
    }
}

}  // namespace gva
