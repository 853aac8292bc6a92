// The projections around the attention of one decode step (Algorithm 1: q_t = x_t W_Q, v_t = x_t W_V,
// k^rope_t = (x_t W_r) R_t^T; then the concatenation of heads and the output projection), with the
// reconstruction maps folded into the query projection offline:  q~_h = x (W_Q^{nope,h} M_h^T)  (Eq. absorb
// applied to the projection), so no separate absorb step remains.
//
// Both are skinny GEMMs  C[M x N] = A[M x K] W[K x N]  with M = batch (tens to hundreds of rows), bf16 weights
// and f32 activations.  One block owns 16 output columns over the whole K: its 16-column slab of W is staged
// once in shared memory with cp.async (48-byte rows: conflict-free for ldmatrix without a swizzle); each warp
// owns a 16-row m-tile and a slice of K (small batches leave most of a block's eight warps without an m-tile
// of their own, so they split K instead and their partial sums meet in shared memory), reads its activations
// straight from global memory in mma A-fragment order, splits every
// f32 activation into three bf16 terms (hi + mid + lo carry all 24 significant bits, so only the weights'
// own bf16 storage limits accuracy) and issues three m16n8k16 MMAs per fragment with f32 accumulation.
// The input projection's epilogue writes the absorbed queries (rotating the positional slice in fp64) and
// appends the new value rows and the rotated positional key to the paged cache.
#pragma once

#include "gva_common.cuh"
#include "gva_small_kernels.cuh"

namespace gva {

constexpr int kProjCols = 16;             // output columns per block
constexpr int kProjRowBytes = 48;         // shared-memory stride of one k-row of the slab (32 bytes used)
constexpr int kProjWarps = 8;             // m-tiles per block: 128 rows

__device__ __forceinline__ void ldsm_x4_trans_p(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_p(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (x, y) -> three packed bf16x2 registers whose element-wise sum reproduces x and y to 24 bits
__device__ __forceinline__ void split3(float x, float y, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(hi) : "f"(y), "f"(x));
    const float rx = x - __uint_as_float(hi << 16), ry = y - __uint_as_float(hi & 0xffff0000u);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(mid) : "f"(ry), "f"(rx));
    const float sx = rx - __uint_as_float(mid << 16), sy = ry - __uint_as_float(mid & 0xffff0000u);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(lo) : "f"(sy), "f"(sx));
}

struct ProjParams {
    const float *A;              // [M][K] activations
    const uint16_t *W;           // [K][N] bf16 weights
    int M, K, N;
    int m_tiles, k_slices;       // per block: m_tiles * k_slices == kProjWarps, K % (16 * k_slices) == 0
    // plain epilogue
    float *Y;                    // [M][N]
    // input-projection epilogue
    float *q_abs;                // [M][H][d_v + d_r]
    void *v_pool, *kr_pool;
    const int32_t *block_table, *pos;
    int32_t *dev_status;
    int H, G, d_v, d_r, P, num_pages, max_pages;
};

// MODE 0: Y = A W.   MODE 1: input projection with the fused query / rotation / append epilogue.
template <int MODE, typename CT>
__global__ void __launch_bounds__(32 * kProjWarps)
project_kernel(ProjParams p, RopeTable rope) {
    grid_dependency_launch();
    extern __shared__ __align__(16) unsigned char slab[];      // [K][48 bytes]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kProjCols;
    const int mt = warp % p.m_tiles, ks = warp / p.m_tiles;
    const int m0 = (blockIdx.y * p.m_tiles + mt) * 16;
    const int k_len = p.K / p.k_slices, k_begin = ks * k_len;
    float *s_red = reinterpret_cast<float *>(slab + (size_t)p.K * kProjRowBytes);      // [kProjWarps][32][8] partial sums
    grid_dependency_wait();
    // stage this block's 16 columns of W: two 16-byte chunks per k-row
    {
        const uint32_t s_u32 = smem_u32(slab);
        const unsigned char *src = reinterpret_cast<const unsigned char *>(p.W);
        for (int c = tid; c < p.K * 2; c += 32 * kProjWarps) {
            const int k = c >> 1, half = c & 1;
            const bool in = n0 + half * 8 < p.N;       // N is a multiple of 8; a block may hang over the last 8 columns
            cp_async16(s_u32 + k * kProjRowBytes + half * 16, src + (in ? ((size_t)k * p.N + n0) * 2 + half * 16 : 0),
                       in ? 16 : 0);
        }
        cp_async_commit();
    }
    const bool warp_live = m0 < p.M;
    const int r_lo = min(m0 + (lane >> 2), p.M - 1), r_hi = min(m0 + (lane >> 2) + 8, p.M - 1);
    const float *a_lo = p.A + (size_t)r_lo * p.K + 2 * (lane & 3);
    const float *a_hi = p.A + (size_t)r_hi * p.K + 2 * (lane & 3);
    float acc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;
    cp_async_wait<0>();
    __syncthreads();
    if (warp_live) {
        // ldmatrix.trans lane addressing: matrices (k0-7, n0-7) (k8-15, n0-7) (k0-7, n8-15) (k8-15, n8-15)
        const uint32_t b_base = smem_u32(slab) + ((lane & 7) + ((lane >> 3) & 1) * 8) * kProjRowBytes + (lane >> 4) * 16;
#pragma unroll 8
        for (int k0 = k_begin; k0 < k_begin + k_len; k0 += 16) {
            const float2 f0 = *reinterpret_cast<const float2 *>(a_lo + k0);
            const float2 f1 = *reinterpret_cast<const float2 *>(a_hi + k0);
            const float2 f2 = *reinterpret_cast<const float2 *>(a_lo + k0 + 8);
            const float2 f3 = *reinterpret_cast<const float2 *>(a_hi + k0 + 8);
            uint32_t ah[4], am[4], al[4], b[4];
            split3(f0.x, f0.y, ah[0], am[0], al[0]);
            split3(f1.x, f1.y, ah[1], am[1], al[1]);
            split3(f2.x, f2.y, ah[2], am[2], al[2]);
            split3(f3.x, f3.y, ah[3], am[3], al[3]);
            ldsm_x4_trans_p(b_base + k0 * kProjRowBytes, b);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                mma_bf16_p(acc[t], al, b[2 * t], b[2 * t + 1]);      // smallest terms first
                mma_bf16_p(acc[t], am, b[2 * t], b[2 * t + 1]);
                mma_bf16_p(acc[t], ah, b[2 * t], b[2 * t + 1]);
            }
        }
    }
    if (p.k_slices > 1) {       // block-uniform: the K slices of an m-tile are summed in slice order by slice 0
        float *mine = s_red + ((size_t)warp * 32 + lane) * 8;
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) mine[t * 4 + e] = acc[t][e];
        __syncthreads();
        if (ks != 0) return;
        for (int s2 = 1; s2 < p.k_slices; ++s2) {
            const float *other = s_red + ((size_t)(s2 * p.m_tiles + mt) * 32 + lane) * 8;
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[t][e] += other[t * 4 + e];
        }
    }
    if (!warp_live) return;
    // ---- epilogue: thread holds rows m0 + lane/4 (+8), columns n0 + t*8 + 2*(lane%4) + {0,1} ----
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const int row = m0 + (lane >> 2) + rr * 8;
        if (row >= p.M) continue;
        if constexpr (MODE == 0) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int n = n0 + t * 8 + 2 * (lane & 3);
                if (n < p.N)
                    *reinterpret_cast<float2 *>(p.Y + (size_t)row * p.N + n) = make_float2(acc[t][2 * rr], acc[t][2 * rr + 1]);
            }
        } else {
            const int dq = p.d_v + p.d_r, nq = p.H * dq, nv = p.G * p.d_v;
            const int t_pos = p.pos[row];
            // cache slot of this sequence's new token (needed only by the value / positional-key columns)
            long long page = -1;
            int slot = 0;
            const bool cache_cols = n0 + kProjCols > nq;
            if (cache_cols) {
                if (t_pos < 0 || t_pos / p.P >= p.max_pages) {
                    if ((lane & 3) == 0) report_error(p.dev_status, GVA_ERR_SEQ_LEN, row);
                } else {
                    page = p.block_table ? (long long)p.block_table[(size_t)row * p.max_pages + t_pos / p.P]
                                         : (long long)row * p.max_pages + t_pos / p.P;
                    if (page < 0 || page >= p.num_pages) {
                        if ((lane & 3) == 0) report_error(p.dev_status, GVA_ERR_BAD_PAGE, row);
                        page = -1;
                    }
                    slot = t_pos % p.P;
                }
            }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int n = n0 + t * 8 + 2 * (lane & 3);
                const float c0 = acc[t][2 * rr], c1 = acc[t][2 * rr + 1];
                if (n >= p.N) continue;
                if (n < nq) {
                    const int h = n / dq, j = n % dq;
                    float *dst = p.q_abs + ((size_t)row * p.H + h) * dq + j;
                    if (j < p.d_v) {
                        *reinterpret_cast<float2 *>(dst) = make_float2(c0, c1);
                    } else {
                        double y0, y1;
                        rope_pair((double)c0, (double)c1, t_pos, rope.inv_freq[(j - p.d_v) >> 1], y0, y1);
                        *reinterpret_cast<float2 *>(dst) = make_float2(__double2float_rn(y0), __double2float_rn(y1));
                    }
                } else if (page >= 0) {
                    if (n < nq + nv) {
                        const int idx = n - nq, g = idx / p.d_v, d = idx % p.d_v;
                        const size_t off = (((size_t)page * p.G + g) * p.P + slot) * p.d_v + d;
                        if constexpr (sizeof(CT) == 2) {
                            reinterpret_cast<uint32_t *>(reinterpret_cast<uint16_t *>(p.v_pool) + off)[0] =
                                (uint32_t)float_to_bf16_bits(c0) | ((uint32_t)float_to_bf16_bits(c1) << 16);
                        } else {
                            *reinterpret_cast<float2 *>(reinterpret_cast<float *>(p.v_pool) + off) = make_float2(c0, c1);
                        }
                    } else {
                        const int i = (n - nq - nv) >> 1;
                        double y0, y1;
                        rope_pair((double)c0, (double)c1, t_pos, rope.inv_freq[i], y0, y1);
                        const size_t off = ((size_t)page * p.P + slot) * p.d_r + 2 * i;
                        if constexpr (sizeof(CT) == 2) {
                            reinterpret_cast<uint32_t *>(reinterpret_cast<uint16_t *>(p.kr_pool) + off)[0] =
                                (uint32_t)double_to_bf16_bits(y0) | ((uint32_t)double_to_bf16_bits(y1) << 16);
                        } else {
                            *reinterpret_cast<float2 *>(reinterpret_cast<float *>(p.kr_pool) + off) =
                                make_float2(__double2float_rn(y0), __double2float_rn(y1));
                        }
                    }
                }
            }
        }
    }
}

}  // namespace gva
