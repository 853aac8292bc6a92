// The O(1)-in-T kernels of a decode step: query absorption (Eq. absorb + query-side RoPE), cache
// append (Algorithm 1's append lines) and the log-sum-exp merge of split-KV partial results.
#pragma once

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

// One pair of y = x R_pos^T in fp64.
__device__ __forceinline__ void rope_pair(double x0, double x1, int pos, double inv_freq, double &y0, double &y1) {
    double s, c;
    sincos((double)pos * inv_freq, &s, &c);
    y0 = x0 * c - x1 * s;
    y1 = x0 * s + x1 * c;
}

// ---- absorb --------------------------------------------------------------------------------------
// grid (H, ceil(B / kAbsorbBatch)), block 128.  M_h is staged once per block in shared memory
// (row stride d_c + 1 floats) and reused for kAbsorbBatch sequences.
constexpr int kAbsorbBatch = 8;

__global__ void __launch_bounds__(128)
absorb_kernel(const float *__restrict__ q_c, const float *__restrict__ q_r, const float *__restrict__ M,
              const int32_t *__restrict__ q_pos, float *__restrict__ q_abs, int B, int H, int d_v, int d_c,
              int d_r, RopeTable rope) {
    extern __shared__ float smem_f[];
    float *sM = smem_f;                            // [d_v][d_c + 1]
    float *sq = smem_f + d_v * (d_c + 1);          // [kAbsorbBatch][d_c]
    const int h = blockIdx.x;
    const int b0 = blockIdx.y * kAbsorbBatch;
    const int nb = min(kAbsorbBatch, B - b0);
    const int tid = threadIdx.x;
    const float *Mh = M + (size_t)h * d_v * d_c;
    for (int i = tid; i < d_v * d_c; i += 128) sM[(i / d_c) * (d_c + 1) + (i % d_c)] = Mh[i];
    for (int i = tid; i < nb * d_c; i += 128) sq[i] = q_c[((size_t)(b0 + i / d_c) * H + h) * d_c + (i % d_c)];
    __syncthreads();
    const int dq = d_v + d_r;
    for (int o = tid; o < nb * d_v; o += 128) {
        const int bb = o / d_v, i = o % d_v;
        const float *mrow = sM + i * (d_c + 1);
        const float *qrow = sq + bb * d_c;
        float acc = 0.f;
        for (int j = 0; j < d_c; ++j) acc = fmaf(qrow[j], mrow[j], acc);
        q_abs[((size_t)(b0 + bb) * H + h) * dq + i] = acc;
    }
    const int half = d_r / 2;
    for (int o = tid; o < nb * half; o += 128) {
        const int bb = o / half, i = o % half;
        const size_t src = ((size_t)(b0 + bb) * H + h) * d_r + 2 * i;
        double y0, y1;
        rope_pair((double)q_r[src], (double)q_r[src + 1], q_pos[b0 + bb], rope.inv_freq[i], y0, y1);
        float *dst = q_abs + ((size_t)(b0 + bb) * H + h) * dq + d_v + 2 * i;
        dst[0] = __double2float_rn(y0);
        dst[1] = __double2float_rn(y1);
    }
}

// ---- append --------------------------------------------------------------------------------------
// grid B, block 128.  Integer page arithmetic, round-to-nearest-even stores, nothing else touched.
template <typename CT>
__global__ void __launch_bounds__(128)
append_kernel(CT *__restrict__ v_pool, CT *__restrict__ kr_pool, const int32_t *__restrict__ block_table,
              const float *__restrict__ v_new, const float *__restrict__ kr_new, const int32_t *__restrict__ pos,
              int G, int d_v, int d_r, int P, int num_pages, int max_pages, int32_t *dev_status, RopeTable rope) {
    const int b = blockIdx.x;
    const int t = pos[b];
    if (t < 0 || t / P >= max_pages) {
        if (threadIdx.x == 0) report_error(dev_status, GVA_ERR_SEQ_LEN, b);
        return;
    }
    const long long page = block_table ? (long long)block_table[(size_t)b * max_pages + t / P]
                                       : (long long)b * max_pages + t / P;
    if (page < 0 || page >= num_pages) {
        if (threadIdx.x == 0) report_error(dev_status, GVA_ERR_BAD_PAGE, b);
        return;
    }
    const int slot = t % P;
    for (int i = threadIdx.x; i < G * d_v; i += 128) {
        const int g = i / d_v, d = i % d_v;
        const float x = v_new[(size_t)b * G * d_v + i];
        const size_t dst = (((size_t)page * G + g) * P + slot) * d_v + d;
        if constexpr (sizeof(CT) == 2) reinterpret_cast<uint16_t *>(v_pool)[dst] = float_to_bf16_bits(x);
        else reinterpret_cast<float *>(v_pool)[dst] = x;
    }
    for (int i = threadIdx.x; i < d_r / 2; i += 128) {
        double y0, y1;
        rope_pair((double)kr_new[(size_t)b * d_r + 2 * i], (double)kr_new[(size_t)b * d_r + 2 * i + 1], t,
                  rope.inv_freq[i], y0, y1);
        const size_t dst = ((size_t)page * P + slot) * d_r + 2 * i;
        if constexpr (sizeof(CT) == 2) {
            reinterpret_cast<uint16_t *>(kr_pool)[dst] = double_to_bf16_bits(y0);
            reinterpret_cast<uint16_t *>(kr_pool)[dst + 1] = double_to_bf16_bits(y1);
        } else {
            reinterpret_cast<float *>(kr_pool)[dst] = __double2float_rn(y0);
            reinterpret_cast<float *>(kr_pool)[dst + 1] = __double2float_rn(y1);
        }
    }
}

// ---- LSE combine ---------------------------------------------------------------------------------
// grid (B, H / 4), block 128: one warp per (sequence, head).  Records are merged in index order, so
// the result is reproducible for fixed launch geometry.
//   m* = max_r m_r ;  L = sum_r l_r 2^(m_r - m*) ;  out = sum_r 2^(m_r - m*) o_r / L ;  lse = (m* + log2 L) ln 2
template <int DV>
__global__ void __launch_bounds__(128)
combine_kernel(DecodeParams p) {
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y * 4 + warp;
    if (h >= p.H) return;
    int first, n;
    if (p.num_splits > 0) {
        first = b * p.num_splits;
        n = p.num_splits;
    } else {
        const int total = p.hdr[0], n_eff = p.hdr[1];
        const int off0 = p.hdr[kHdrInts + b], off1 = p.hdr[kHdrInts + b + 1];
        if (off1 == off0) {
            n = 0;
            first = 0;
        } else {
            const int c0 = range_owner(off0, total, n_eff), c1 = range_owner(off1 - 1, total, n_eff);
            first = c0 + b;
            n = c1 - c0 + 1;
        }
    }
    constexpr int DPL = DV / 32;
    float *o_dst = p.out + ((size_t)b * p.H + h) * DV + lane * DPL;
    float mstar = -INFINITY;
    for (int r = lane; r < n; r += 32) mstar = fmaxf(mstar, p.rec_ml[((size_t)(first + r) * p.H + h) * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, o));
    if (n == 0 || mstar == -INFINITY) {
#pragma unroll
        for (int d = 0; d < DPL; ++d) o_dst[d] = 0.f;
        if (p.lse && lane == 0) p.lse[(size_t)b * p.H + h] = -INFINITY;
        return;
    }
    float L = 0.f, acc[DPL];
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[d] = 0.f;
    for (int r = 0; r < n; ++r) {
        const size_t rh = (size_t)(first + r) * p.H + h;
        const float2 ml = *reinterpret_cast<const float2 *>(p.rec_ml + rh * 2);
        if (ml.x == -INFINITY) continue;   // empty partition: weight 0
        const float w = exp2f(ml.x - mstar);
        L = fmaf(ml.y, w, L);
        const float *o = p.rec_o + rh * DV + lane * DPL;
        if constexpr (DPL == 2) {
            const float2 v = *reinterpret_cast<const float2 *>(o);
            acc[0] = fmaf(w, v.x, acc[0]);
            acc[1] = fmaf(w, v.y, acc[1]);
        } else {
            const float4 v = *reinterpret_cast<const float4 *>(o);
            acc[0] = fmaf(w, v.x, acc[0]);
            acc[1] = fmaf(w, v.y, acc[1]);
            acc[2] = fmaf(w, v.z, acc[2]);
            acc[3] = fmaf(w, v.w, acc[3]);
        }
    }
    const float inv = 1.f / L;
#pragma unroll
    for (int d = 0; d < DPL; ++d) o_dst[d] = acc[d] * inv;
    if (p.lse && lane == 0) p.lse[(size_t)b * p.H + h] = (mstar + log2f(L)) * kLn2;
}

}  // namespace gva
