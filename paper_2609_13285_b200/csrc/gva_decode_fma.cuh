// CUDA-core (FMA) split-KV decode kernel over the paged GVA cache.
//
// One thread block owns a contiguous range of 32-token tiles of the batch's cache stream; one warp
// per value group.  Tiles are staged global->shared with 16-byte cp.async copies in a ring of
// NSTAGE buffers (rows padded by 16 bytes so that both access patterns below are conflict-free):
//   scores : lane = token.  s_h = q~_h . v_t + q^rope_h . k^rope_t for the group's 4 heads, the
//            absorbed query read from shared memory as broadcast float4.
//   softmax: online, base 2 (scale * log2 e folded into the scores), warp-shuffle max; the running
//            sum is kept per lane and reduced once per segment.
//   P.V    : lane = value dimensions.  p_t of the 4 heads broadcast from shared memory.
// This kernel serves the f32 cache (exact f32 arithmetic end to end) and is the CUDA-core
// baseline for the bf16 cache.
#pragma once

#include "gva_common.cuh"

namespace gva {

template <typename CT, int DV, int DR, bool GQA>
struct FmaTraits {
    static constexpr int TILE = 32;
    static constexpr int EPC = 16 / (int)sizeof(CT);           // elements per 16-byte chunk
    static constexpr int VROW = DV * (int)sizeof(CT) + 16;      // padded value (and GQA key) row, bytes
    static constexpr int KROW = DR * (int)sizeof(CT) + 16;      // padded positional-key row, bytes
    static constexpr int VCH = DV / EPC;
    static constexpr int KCH = DR / EPC;
    static constexpr int DQ = GQA ? DV : DV + DR;               // query width
    static constexpr int DPL = DV / 32;                         // value dims per lane in P.V
    // bytes of one stage for G groups: GVA = G value tiles + 1 positional tile; GQA = G key + G value tiles
    __host__ __device__ static constexpr int stage_bytes(int G) {
        return GQA ? 2 * G * TILE * VROW : G * TILE * VROW + TILE * KROW;
    }
    __host__ __device__ static constexpr int fixed_bytes(int B, int H, int G) {
        // tile offsets, query, P exchange, per-stage valid counts
        return (((B + 1) * 4 + 15) & ~15) + H * DQ * 4 + G * TILE * 16 + 64;
    }
};

template <typename CT, int N>
__device__ __forceinline__ void unpack_chunk(const uint4 &raw, float (&v)[N]) {
    if constexpr (sizeof(CT) == 2) {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else {
        v[0] = __uint_as_float(raw.x);
        v[1] = __uint_as_float(raw.y);
        v[2] = __uint_as_float(raw.z);
        v[3] = __uint_as_float(raw.w);
    }
}

template <typename CT, int DV, int DR, bool GQA, int NSTAGE>
__global__ void __launch_bounds__(256)
decode_fma_kernel(DecodeParams p) {
    using T = FmaTraits<CT, DV, DR, GQA>;
    constexpr int TILE = T::TILE;
    grid_dependency_launch();
    extern __shared__ __align__(16) unsigned char smem[];
    const int G = p.G, H = p.H;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int warp = tid >> 5, lane = tid & 31;   // warp == value group

    int *s_off = reinterpret_cast<int *>(smem);
    float *sQ = reinterpret_cast<float *>(smem + (((p.B + 1) * 4 + 15) & ~15));
    float4 *sP = reinterpret_cast<float4 *>(sQ + H * T::DQ);           // [G][TILE]
    int *s_nvalid = reinterpret_cast<int *>(sP + G * TILE);            // [NSTAGE] (<= 16)
    unsigned char *stages = reinterpret_cast<unsigned char *>(s_nvalid) + 64;
    const int stage_bytes = T::stage_bytes(G);

    grid_dependency_wait();
    compute_tile_offsets<TILE>(p, s_off);
    const UnitPlan plan = make_unit_plan(s_off[p.B], gridDim.x, false);     // one unit per block: unit id = block index
    block0_duties(p, s_off, plan, tid, nt);
    const BlockRange rg = block_range(p, s_off);
    const int n_tiles = rg.hi - rg.lo;

    if (n_tiles <= 0) {
        // uniform mode: an empty split still owns a record (weight 0 in the merge)
        if (rg.rec_fixed >= 0) {
            for (int i = tid; i < H; i += nt) {
                p.rec_ml[((size_t)rg.rec_fixed * H + i) * 2] = -INFINITY;
                p.rec_ml[((size_t)rg.rec_fixed * H + i) * 2 + 1] = 0.f;
            }
        }
        return;
    }

    // ---- tile loader: flat tile f of this block -> (sequence, tile in sequence) -> cp.async copies
    int ld_b = rg.b_first;   // cursor of the loader (runs NSTAGE-1 tiles ahead of the consumer)
    auto issue_tile = [&](int i) {
        const int f = rg.lo + i;
        while (f >= s_off[ld_b + 1]) ++ld_b;
        const int b = ld_b;
        const int t0 = (f - s_off[b]) * TILE;
        int n_valid = min(TILE, p.seq_lens[b] - t0);
        const int pj = t0 / p.P, slot0 = t0 % p.P;
        long long page = p.block_table ? (long long)p.block_table[(size_t)b * p.max_pages + pj]
                                       : (long long)b * p.max_pages + pj;
        if (page < 0 || page >= p.num_pages) {
            if (tid == 0) report_error(p.dev_status, GVA_ERR_BAD_PAGE, b);
            page = 0;
            n_valid = 0;
        }
        unsigned char *st = stages + (size_t)(i % NSTAGE) * stage_bytes;
        if (tid == 0) s_nvalid[i % NSTAGE] = n_valid;
        const uint32_t st_u32 = smem_u32(st);
        const int n_vchunks = G * TILE * T::VCH;
        const unsigned char *vsrc = reinterpret_cast<const unsigned char *>(p.v_pool);
        for (int c = tid; c < n_vchunks; c += nt) {
            const int ch = c % T::VCH, t = (c / T::VCH) % TILE, g = c / (T::VCH * TILE);
            const size_t row = ((size_t)page * G + g) * p.P + slot0 + t;
            const int ok = t < n_valid;
            cp_async16(st_u32 + (g * TILE + t) * T::VROW + ch * 16,
                       vsrc + (ok ? row * (DV * sizeof(CT)) + ch * 16 : 0), ok ? 16 : 0);
        }
        if constexpr (GQA) {
            const unsigned char *ksrc = reinterpret_cast<const unsigned char *>(p.k_pool);
            const uint32_t kb = st_u32 + G * TILE * T::VROW;
            for (int c = tid; c < n_vchunks; c += nt) {
                const int ch = c % T::VCH, t = (c / T::VCH) % TILE, g = c / (T::VCH * TILE);
                const size_t row = ((size_t)page * G + g) * p.P + slot0 + t;
                const int ok = t < n_valid;
                cp_async16(kb + (g * TILE + t) * T::VROW + ch * 16,
                           ksrc + (ok ? row * (DV * sizeof(CT)) + ch * 16 : 0), ok ? 16 : 0);
            }
        } else if constexpr (DR > 0) {      // (the value-only cache has no positional tile)
            const unsigned char *ksrc = reinterpret_cast<const unsigned char *>(p.kr_pool);
            const uint32_t kb = st_u32 + G * TILE * T::VROW;
            for (int c = tid; c < TILE * T::KCH; c += nt) {
                const int ch = c % T::KCH, t = c / T::KCH;
                const size_t row = (size_t)page * p.P + slot0 + t;
                const int ok = t < n_valid;
                cp_async16(kb + t * T::KROW + ch * 16, ksrc + (ok ? row * (DR * sizeof(CT)) + ch * 16 : 0),
                           ok ? 16 : 0);
            }
        }
    };

    if constexpr (NSTAGE > 1) {
#pragma unroll 1
        for (int i = 0; i < NSTAGE - 1; ++i) {
            if (i < n_tiles) issue_tile(i);
            cp_async_commit();
        }
    }

    // ---- consumer state (per warp = group, 4 heads) ----
    float m_run[4], l_run[4], acc[4][T::DPL];
    int cur_b = -1;
    int cs_b = rg.b_first;   // consumer cursor

#pragma unroll 1
    for (int i = 0; i < n_tiles; ++i) {
        if constexpr (NSTAGE > 1) {
            cp_async_wait<NSTAGE - 2>();
            __syncthreads();
            if (i + NSTAGE - 1 < n_tiles) issue_tile(i + NSTAGE - 1);
            cp_async_commit();
        } else {
            __syncthreads();
            issue_tile(i);
            cp_async_commit();
            cp_async_wait<0>();
            __syncthreads();
        }
        const int f = rg.lo + i;
        while (f >= s_off[cs_b + 1]) ++cs_b;
        const int b = cs_b;
        if (b != cur_b) {   // new segment: stage this sequence's queries, reset the softmax state
            cur_b = b;
            const float *qsrc = p.q + (size_t)b * H * T::DQ;
            for (int k = tid; k < H * T::DQ; k += nt) sQ[k] = qsrc[k];
            __syncthreads();
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                m_run[h] = -INFINITY;
                l_run[h] = 0.f;
#pragma unroll
                for (int d = 0; d < T::DPL; ++d) acc[h][d] = 0.f;
            }
        }
        const unsigned char *st = stages + (size_t)(i % NSTAGE) * stage_bytes;
        const int n_valid = s_nvalid[i % NSTAGE];
        const unsigned char *vt = st + (size_t)warp * TILE * T::VROW;
        const float *q0 = sQ + (size_t)(warp * kHeadsPerGroup) * T::DQ;

        // scores, lane = token
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const unsigned char *krow_base = GQA ? st + (size_t)(G + warp) * TILE * T::VROW : vt;
            const unsigned char *row = krow_base + lane * T::VROW;   // GVA: the value row is the content key source
#pragma unroll
            for (int c = 0; c < T::VCH; ++c) {
                float v[T::EPC];
                unpack_chunk<CT>(*reinterpret_cast<const uint4 *>(row + c * 16), v);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float *qh = q0 + h * T::DQ + c * T::EPC;
#pragma unroll
                    for (int e = 0; e < T::EPC; e += 4) {
                        const float4 q4 = *reinterpret_cast<const float4 *>(qh + e);
                        s[h] = fmaf(q4.x, v[e], s[h]);
                        s[h] = fmaf(q4.y, v[e + 1], s[h]);
                        s[h] = fmaf(q4.z, v[e + 2], s[h]);
                        s[h] = fmaf(q4.w, v[e + 3], s[h]);
                    }
                }
            }
            if constexpr (!GQA) {
                const unsigned char *krow = st + (size_t)G * TILE * T::VROW + lane * T::KROW;
#pragma unroll
                for (int c = 0; c < T::KCH; ++c) {
                    float v[T::EPC];
                    unpack_chunk<CT>(*reinterpret_cast<const uint4 *>(krow + c * 16), v);
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const float *qh = q0 + h * T::DQ + DV + c * T::EPC;
#pragma unroll
                        for (int e = 0; e < T::EPC; e += 4) {
                            const float4 q4 = *reinterpret_cast<const float4 *>(qh + e);
                            s[h] = fmaf(q4.x, v[e], s[h]);
                            s[h] = fmaf(q4.y, v[e + 1], s[h]);
                            s[h] = fmaf(q4.z, v[e + 2], s[h]);
                            s[h] = fmaf(q4.w, v[e + 3], s[h]);
                        }
                    }
                }
            }
        }
        // online softmax (base 2)
        float pr[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const float sc = (lane < n_valid) ? s[h] * p.scale_log2 : -INFINITY;
            float tmax = sc;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            const float m_new = fmaxf(m_run[h], tmax);
            float corr = 1.f;
            pr[h] = 0.f;
            if (m_new != -INFINITY) {
                corr = exp2f(m_run[h] - m_new);
                pr[h] = exp2f(sc - m_new);
            }
            m_run[h] = m_new;
            l_run[h] = fmaf(l_run[h], corr, pr[h]);
#pragma unroll
            for (int d = 0; d < T::DPL; ++d) acc[h][d] *= corr;
        }
        __syncwarp();
        sP[warp * TILE + lane] = make_float4(pr[0], pr[1], pr[2], pr[3]);
        __syncwarp();
        // P.V, lane = value dims [lane*DPL, lane*DPL + DPL)
#pragma unroll 8
        for (int t = 0; t < TILE; ++t) {
            const float4 p4 = sP[warp * TILE + t];
            const unsigned char *vr = vt + t * T::VROW + lane * (T::DPL * (int)sizeof(CT));
            float v[T::DPL];
            if constexpr (sizeof(CT) == 2 && T::DPL == 2) {
                const uint32_t w = *reinterpret_cast<const uint32_t *>(vr);
                v[0] = __uint_as_float(w << 16);
                v[1] = __uint_as_float(w & 0xffff0000u);
            } else if constexpr (sizeof(CT) == 2 && T::DPL == 4) {
                const uint2 w = *reinterpret_cast<const uint2 *>(vr);
                v[0] = __uint_as_float(w.x << 16);
                v[1] = __uint_as_float(w.x & 0xffff0000u);
                v[2] = __uint_as_float(w.y << 16);
                v[3] = __uint_as_float(w.y & 0xffff0000u);
            } else if constexpr (T::DPL == 2) {
                const float2 w = *reinterpret_cast<const float2 *>(vr);
                v[0] = w.x;
                v[1] = w.y;
            } else {
                const float4 w = *reinterpret_cast<const float4 *>(vr);
                v[0] = w.x;
                v[1] = w.y;
                v[2] = w.z;
                v[3] = w.w;
            }
#pragma unroll
            for (int d = 0; d < T::DPL; ++d) {
                acc[0][d] = fmaf(p4.x, v[d], acc[0][d]);
                acc[1][d] = fmaf(p4.y, v[d], acc[1][d]);
                acc[2][d] = fmaf(p4.z, v[d], acc[2][d]);
                acc[3][d] = fmaf(p4.w, v[d], acc[3][d]);
            }
        }
        // segment end: this block's range ends or the next tile belongs to another sequence
        if (i + 1 == n_tiles || f + 1 >= s_off[b + 1]) {
            const int rec = (rg.rec_fixed >= 0) ? rg.rec_fixed : (int)blockIdx.x + b;
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                float l = l_run[h];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                const size_t rh = (size_t)rec * H + warp * kHeadsPerGroup + h;
                float *o_dst = p.rec_o + rh * DV + lane * T::DPL;
#pragma unroll
                for (int d = 0; d < T::DPL; ++d) o_dst[d] = acc[h][d];
                if (lane == 0) {
                    p.rec_ml[rh * 2] = m_run[h];
                    p.rec_ml[rh * 2 + 1] = l;
                }
            }
        }
    }
    cp_async_wait<0>();
}

}  // namespace gva
