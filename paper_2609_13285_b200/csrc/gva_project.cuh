// The projections around the attention of one decode step (Algorithm 1: q_t = x_t W_Q, v_t = x_t W_V,
// k^rope_t = (x_t W_r) R_t^T; then the concatenation of heads and the output projection), with the
// reconstruction maps folded into the query projection offline:  q~_h = x (W_Q^{nope,h} M_h^T)  (Eq. absorb
// applied to the projection), so no separate absorb step remains.
//
// Both are skinny GEMMs  C[M x N] = A[M x K] W[K x N]  with M = batch (tens to hundreds of rows), bf16 weights
// and f32 activations: too few rows to fill the machine by output tiles alone, so K is split eight ways across
// a thread-block cluster.  Block (n, r) of a cluster computes the partial product of a 64-column strip over
// K-slice r: its slice of W (K/8 rows of 128 contiguous bytes) is staged with cp.async into 144-byte rows
// (conflict-free for ldmatrix without a swizzle); each warp owns a 16-row m-tile and some of the strip's eight
// n-tiles, reads its activations straight from global memory in mma A-fragment order, splits every f32
// activation into three bf16 terms (hi + mid + lo carry all 24 significant bits, so only the weights' own bf16
// storage limits accuracy) and issues three m16n8k16 MMAs per fragment with f32 accumulation.  The partial
// strips meet through distributed shared memory: after a cluster barrier block r sums columns [8r, 8r + 8) of
// all eight partials in rank order (deterministic) and runs the epilogue for them.  The input projection's
// epilogue writes the absorbed queries (rotating the positional slice in fp64) and appends the new value rows
// and the rotated positional key to the paged cache.
#pragma once

#include <cooperative_groups.h>

#include "gva_common.cuh"
#include "gva_small_kernels.cuh"

namespace gva {

namespace cg = cooperative_groups;

constexpr int kProjStrip = 64;            // output columns per cluster
constexpr int kProjSlices = 8;            // K slices = blocks per cluster
constexpr int kProjRowBytes = 144;        // shared-memory stride of one k-row of the W slice (128 bytes used)
constexpr int kProjWarps = 8;             // 256 threads
constexpr int kProjRows = 128;            // rows (sequences) per block
constexpr int kProjLd = kProjStrip + 4;   // f32 row stride of the partial strip in shared memory

__device__ __forceinline__ void ldsm_x2_trans_p(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];\n" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
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
    // plain epilogue
    float *Y;                    // [M][N]
    // input-projection epilogue
    float *q_abs;                // [M][H][d_v + d_r]
    void *v_pool, *kr_pool;
    const int32_t *block_table, *pos;
    int32_t *dev_status;
    int H, G, d_v, d_r, P, num_pages, max_pages;
};

// One finished pair of outputs (row, columns n and n + 1).
// MODE 0: Y = A W.   MODE 1: input projection: absorbed query / rotated positional query / value append / rotated key append.
template <int MODE, typename CT>
__device__ __forceinline__ void project_epilogue(const ProjParams &p, const RopeTable &rope, int row, int n, float c0, float c1,
                                                 int t_pos) {
    if constexpr (MODE == 0) {
        *reinterpret_cast<float2 *>(p.Y + (size_t)row * p.N + n) = make_float2(c0, c1);
    } else {
        const int dq = p.d_v + p.d_r, nq = p.H * dq, nv = p.G * p.d_v;
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
            return;
        }
        // cache slot of this sequence's new token; one thread per (row, strip) reports a bad position
        const bool reporter = (n & (kProjStrip - 1)) == 0 || n == nq;
        if (t_pos < 0 || t_pos / p.P >= p.max_pages) {
            if (reporter) report_error(p.dev_status, GVA_ERR_SEQ_LEN, row);
            return;
        }
        const long long page = p.block_table ? (long long)p.block_table[(size_t)row * p.max_pages + t_pos / p.P]
                                             : (long long)row * p.max_pages + t_pos / p.P;
        if (page < 0 || page >= p.num_pages) {
            if (reporter) report_error(p.dev_status, GVA_ERR_BAD_PAGE, row);
            return;
        }
        const int slot = t_pos % p.P;
        if (n < nq + nv) {
            const int idx = n - nq, g = idx / p.d_v, d = idx % p.d_v;
            const size_t off = (((size_t)page * p.G + g) * p.P + slot) * p.d_v + d;
            if constexpr (sizeof(CT) == 1) {
                reinterpret_cast<uint16_t *>(reinterpret_cast<uint8_t *>(p.v_pool) + off)[0] =
                    (uint16_t)((uint32_t)float_to_e4m3_bits(c0) | ((uint32_t)float_to_e4m3_bits(c1) << 8));
            } else if constexpr (sizeof(CT) == 2) {
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
            if constexpr (sizeof(CT) == 1) {
                reinterpret_cast<uint16_t *>(reinterpret_cast<uint8_t *>(p.kr_pool) + off)[0] =
                    (uint16_t)((uint32_t)double_to_e4m3_bits(y0) | ((uint32_t)double_to_e4m3_bits(y1) << 8));
            } else if constexpr (sizeof(CT) == 2) {
                reinterpret_cast<uint32_t *>(reinterpret_cast<uint16_t *>(p.kr_pool) + off)[0] =
                    (uint32_t)double_to_bf16_bits(y0) | ((uint32_t)double_to_bf16_bits(y1) << 16);
            } else {
                *reinterpret_cast<float2 *>(reinterpret_cast<float *>(p.kr_pool) + off) =
                    make_float2(__double2float_rn(y0), __double2float_rn(y1));
            }
        }
    }
}

// grid (ceil(N / 64), 8, ceil(M / 128)), cluster (1, 8, 1), block 256.
// MT = m-tiles per block (power of two); 8 / MT warps share an m-tile and each takes MT of the strip's 8 n-tiles.
// The K slice is walked in chunks of 128: the chunk of W and the chunk of activations are both staged with
// cp.async (one memory round trip per chunk) and the k-steps run as a small rolled loop over shared memory --
// short kernels like this one are dominated by instruction fetch when their code is large, because the cache
// stream between two calls pushes it out of L2.
constexpr int kProjChunk = 128;                       // k per staged chunk
constexpr int kProjALd = kProjChunk + 8;              // f32 row stride of the staged activations (conflict-free float2 reads)

template <int MODE, typename CT, int MT>
__global__ void __launch_bounds__(32 * kProjWarps)
project_kernel(ProjParams p, RopeTable rope) {
    // The input projection lets its dependent (the decode kernel of a layer step) start only once it has itself waited
    // for everything earlier in the stream, as step_front_kernel does: what that kernel does ahead of its own wait then
    // overlaps with this kernel only.  The output projection has no such follower and releases its dependent at once.
    if constexpr (MODE != 1) grid_dependency_launch();
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) unsigned char psm[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k_len = p.K / kProjSlices;
    unsigned char *w_s = psm;                                                        // [kProjChunk][144 bytes]
    float *a_s = reinterpret_cast<float *>(psm + (size_t)kProjChunk * kProjRowBytes);  // [16 MT][kProjALd]
    float *part = a_s;                                                               // [16 MT][kProjLd], after the last chunk
    const int n0 = blockIdx.x * kProjStrip;
    const int rank = blockIdx.y;                  // == cluster rank: the cluster spans y
    const int k_begin = rank * k_len;
    const int row0 = blockIdx.z * kProjRows;
    const int rows = min(kProjRows, p.M - row0);
    const int mt = warp % MT, ng = warp / MT;
    const int m0 = mt * 16;
    const uint32_t w_u32 = smem_u32(w_s), a_u32 = smem_u32(a_s);
    auto request_w = [&](int kc, int kn) {                              // W chunk: kn rows of 8 x 16 bytes
        const unsigned char *src = reinterpret_cast<const unsigned char *>(p.W);
        for (int c = tid; c < kn * 8; c += 32 * kProjWarps) {
            const int k = c >> 3, ch = c & 7;
            const bool in = n0 + ch * 8 < p.N;                         // columns past N read as zero
            cp_async16(w_u32 + k * kProjRowBytes + ch * 16,
                       src + (in ? ((size_t)(k_begin + kc + k) * p.N + n0 + ch * 8) * 2 : 0), in ? 16 : 0);
        }
    };
    // The weights do not come from the work that precedes this kernel in the stream: their first chunk is requested
    // ahead of the wait for that work, so that its round trip overlaps with the end of the preceding kernel.
    request_w(0, min(kProjChunk, k_len));
    grid_dependency_wait();
    if constexpr (MODE == 1) grid_dependency_launch();
    // the epilogue's position lookups travel with the first chunk
    int ep_pos[2] = {0, 0};
    if constexpr (MODE == 1) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int item = tid + u * 32 * kProjWarps;
            if (item < rows * 4) ep_pos[u] = p.pos[row0 + (item >> 2)];
        }
    }
    float acc[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;
    // ldmatrix.x2.trans lane addressing: matrices (k0-7, n-tile) and (k8-15, n-tile); lanes 16-31 repeat 0-15
    const uint32_t b_base = w_u32 + (lane & 15) * kProjRowBytes + ng * MT * 16;
    const float *a_lo = a_s + (m0 + (lane >> 2)) * kProjALd + 2 * (lane & 3);
    const float *a_hi = a_lo + 8 * kProjALd;
#pragma unroll 1
    for (int kc = 0; kc < k_len; kc += kProjChunk) {
        const int kn = min(kProjChunk, k_len - kc);
        if (kc > 0) __syncthreads();              // everyone is done with the previous chunk
        {
            if (kc > 0) request_w(kc, kn);
            const int cpr = kn >> 2;                                    // 16-byte chunks per activation row
            for (int c = tid; c < 16 * MT * cpr; c += 32 * kProjWarps) {
                const int r = c / cpr, ch = c % cpr;
                const int row = row0 + min(r, rows - 1);                // rows past M repeat the last one (never stored)
                cp_async16(a_u32 + (r * kProjALd + ch * 4) * 4, p.A + (size_t)row * p.K + k_begin + kc + ch * 4, 16);
            }
            cp_async_commit();
        }
        cp_async_wait<0>();
        __syncthreads();
#pragma unroll 1
        for (int k0 = 0; k0 < kn; k0 += 16) {
            const float2 f0 = *reinterpret_cast<const float2 *>(a_lo + k0);
            const float2 f1 = *reinterpret_cast<const float2 *>(a_hi + k0);
            const float2 f2 = *reinterpret_cast<const float2 *>(a_lo + k0 + 8);
            const float2 f3 = *reinterpret_cast<const float2 *>(a_hi + k0 + 8);
            uint32_t ah[4], am[4], al[4];
            split3(f0.x, f0.y, ah[0], am[0], al[0]);
            split3(f1.x, f1.y, ah[1], am[1], al[1]);
            split3(f2.x, f2.y, ah[2], am[2], al[2]);
            split3(f3.x, f3.y, ah[3], am[3], al[3]);
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                uint32_t b[2];
                ldsm_x2_trans_p(b_base + k0 * kProjRowBytes + t * 16, b);
                mma_bf16_p(acc[t], al, b[0], b[1]);      // smallest terms first
                mma_bf16_p(acc[t], am, b[0], b[1]);
                mma_bf16_p(acc[t], ah, b[0], b[1]);
            }
        }
    }
    __syncthreads();      // the activation buffer becomes the partial strip
    // partial strip of this K slice: rows m0 + lane/4 (+8), columns (ng*MT + t)*8 + 2*(lane%4) + {0,1}
#pragma unroll
    for (int t = 0; t < MT; ++t) {
        const int col = (ng * MT + t) * 8 + 2 * (lane & 3);
        *reinterpret_cast<float2 *>(part + (m0 + (lane >> 2)) * kProjLd + col) = make_float2(acc[t][0], acc[t][1]);
        *reinterpret_cast<float2 *>(part + (m0 + (lane >> 2) + 8) * kProjLd + col) = make_float2(acc[t][2], acc[t][3]);
    }
    cluster.sync();
    // block `rank` finishes columns [8 rank, 8 rank + 8) of the strip: sum the eight partials in rank order
    const float *remote[kProjSlices];
#pragma unroll
    for (int q = 0; q < kProjSlices; ++q) remote[q] = cluster.map_shared_rank(part, q);
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int item = tid + u * 32 * kProjWarps;     // rows <= 128: at most two items per thread
        if (item >= rows * 4) continue;
        const int r = item >> 2, col = rank * 8 + (item & 3) * 2;
        const int n = n0 + col;
        if (n >= p.N) continue;
        float c0 = 0.f, c1 = 0.f;
#pragma unroll
        for (int q = 0; q < kProjSlices; ++q) {
            const float2 v = *reinterpret_cast<const float2 *>(remote[q] + r * kProjLd + col);
            c0 += v.x;
            c1 += v.y;
        }
        project_epilogue<MODE, CT>(p, rope, row0 + r, n, c0, c1, ep_pos[u]);
    }
    cluster.sync();      // nobody leaves while another block may still read its shared memory
}

}  // namespace gva
