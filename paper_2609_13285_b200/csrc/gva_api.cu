// Host side of the C ABI declared in include/gva.h: argument validation, launch geometry, kernel
// dispatch.  No device memory is allocated here and no call synchronises.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <mutex>
#include <new>

#include "gva_common.cuh"
#include "gva_decode_fma.cuh"
#include "gva_small_kernels.cuh"
#include "gva_project.cuh"
#ifdef GVA_WITH_MMA
#include "gva_decode_mma.cuh"
#include "gva_decode_fp8.cuh"
#include "gva_prefill.cuh"
#endif

using namespace gva;

struct gva_handle {
    gva_config cfg;
    int device;
    int sm_count;
    int smem_optin;          // max dynamic shared memory per block
    int smem_per_sm;         // shared memory of one SM
    float scale;             // softmax scale of gva_decode
    RopeTable rope;
    int last_num_splits;
    int last_kernel;
    int last_tile;
    int epoch;               // number of the last decode call on this handle (see kSync* in gva_common.cuh)
    int serial;              // number of this handle among all created in this process (see kHdrEpoch)
    int32_t *sync_base;      // device address of the sync arena on this handle's device
    int sync_off, sync_cap;  // the region of the arena in use (words)
    int n_regions;           // regions reserved so far (the earlier, smaller ones are kept until gva_destroy)
    int region_off[24], region_cap[24];
#ifdef GVA_WITH_MMA
    MmaHostState mma;
#endif
};

// ---- device-side scheduling state ------------------------------------------------------------------
// The decode and combine kernels coordinate through a few int32 words per handle (gva_common.cuh, kSync*): the tickets
// that hand out tail units and the per-sequence arrival counters the combine kernel polls.  They live in an arena
// inside the library image (zero at load), so no caller buffer has to be initialised and no caller can overwrite them;
// a handle reserves a region of it sized for its largest batch so far.  Calls on one handle are stream-ordered by
// contract, so a region has one user at a time.
constexpr int kSyncArenaInts = 1 << 20;          // 4 MiB of device memory per GPU that loads the library
static __device__ int32_t g_sync_arena[kSyncArenaInts];

namespace {
std::mutex g_arena_mutex;
struct FreeRange { int off, len; };
constexpr int kMaxFreeRanges = 4096;
FreeRange g_free[kMaxFreeRanges] = {{0, kSyncArenaInts}};
int g_n_free = 1;

// first fit; -1 when the arena is exhausted
int arena_reserve(int len) {
    std::lock_guard<std::mutex> lock(g_arena_mutex);
    for (int i = 0; i < g_n_free; ++i)
        if (g_free[i].len >= len) {
            const int off = g_free[i].off;
            g_free[i].off += len;
            g_free[i].len -= len;
            if (g_free[i].len == 0) {
                for (int j = i + 1; j < g_n_free; ++j) g_free[j - 1] = g_free[j];
                --g_n_free;
            }
            return off;
        }
    return -1;
}
void arena_release(int off, int len) {
    std::lock_guard<std::mutex> lock(g_arena_mutex);
    int i = 0;
    while (i < g_n_free && g_free[i].off < off) ++i;
    if (g_n_free >= kMaxFreeRanges) return;             // table of holes full: the range is dropped (lost until the library is reloaded)
    for (int j = g_n_free; j > i; --j) g_free[j] = g_free[j - 1];
    g_free[i] = FreeRange{off, len};
    ++g_n_free;
    if (i + 1 < g_n_free && g_free[i].off + g_free[i].len == g_free[i + 1].off) {       // merge with the next hole
        g_free[i].len += g_free[i + 1].len;
        for (int j = i + 2; j < g_n_free; ++j) g_free[j - 1] = g_free[j];
        --g_n_free;
    }
    if (i > 0 && g_free[i - 1].off + g_free[i - 1].len == g_free[i].off) {               // ... and with the previous one
        g_free[i - 1].len += g_free[i].len;
        for (int j = i + 1; j < g_n_free; ++j) g_free[j - 1] = g_free[j];
        --g_n_free;
    }
}

// Makes sure the handle's region holds `need` words; a new, larger region is cleared on `stream` before first use.
int ensure_sync(gva_handle *h, int need, cudaStream_t stream) {
    if (need <= h->sync_cap) return GVA_OK;
    if (h->n_regions >= 24) return GVA_ERR_UNSUPPORTED;
    int cap = 64;
    while (cap < need) cap *= 2;
    const int off = arena_reserve(cap);
    if (off < 0) return GVA_ERR_UNSUPPORTED;            // too many live handles with very large batches
    if (cudaMemsetAsync(h->sync_base + off, 0, (size_t)cap * sizeof(int32_t), stream) != cudaSuccess) {
        (void)cudaGetLastError();
        arena_release(off, cap);
        return GVA_ERR_CUDA;
    }
    h->region_off[h->n_regions] = off;
    h->region_cap[h->n_regions] = cap;
    ++h->n_regions;
    h->sync_off = off;
    h->sync_cap = cap;
    return GVA_OK;
}
}  // namespace

namespace {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- FMA kernel dispatch ---------------------------------------------------------------------
using KernelFn = void (*)(DecodeParams);

template <typename CT, int DV, int DR, bool GQA>
KernelFn fma_kernel_for(int nstage) {
    switch (nstage) {
        case 1: return decode_fma_kernel<CT, DV, DR, GQA, 1>;
        case 2: return decode_fma_kernel<CT, DV, DR, GQA, 2>;
        default: return decode_fma_kernel<CT, DV, DR, GQA, 3>;
    }
}

struct FmaPlan {
    KernelFn fn;
    int nstage;
    size_t smem;
    int threads;
};

template <typename CT, int DV, int DR, bool GQA>
bool plan_fma_t(const gva_handle *h, int B, FmaPlan *out) {
    using T = FmaTraits<CT, DV, DR, GQA>;
    const int G = h->cfg.G, H = h->cfg.H;
    const size_t fixed = T::fixed_bytes(B, H, G);
    const size_t stage = T::stage_bytes(G);
    int nstage = 3;
    // three stages when that still leaves room for three blocks per SM, else two, else one
    if (fixed + 3 * stage > (size_t)h->smem_optin / 3) nstage = 2;
    if (fixed + (size_t)nstage * stage > (size_t)h->smem_optin) nstage = 1;
    if (fixed + (size_t)nstage * stage > (size_t)h->smem_optin) return false;
    out->fn = fma_kernel_for<CT, DV, DR, GQA>(nstage);
    out->nstage = nstage;
    out->smem = fixed + (size_t)nstage * stage;
    out->threads = 32 * G;
    return true;
}

template <bool GQA>
bool plan_fma(const gva_handle *h, int B, FmaPlan *out) {
    const bool bf = h->cfg.cache_dtype == GVA_BF16;
    if (h->cfg.d_v == 64 && h->cfg.d_r == 24 && !GQA)
        return bf ? plan_fma_t<__nv_bfloat16, 64, 24, false>(h, B, out) : plan_fma_t<float, 64, 24, false>(h, B, out);
    if (h->cfg.d_r == 0 && !GQA) {      // value-only cache
        if (h->cfg.d_v == 64) return bf ? plan_fma_t<__nv_bfloat16, 64, 0, false>(h, B, out) : plan_fma_t<float, 64, 0, false>(h, B, out);
        return bf ? plan_fma_t<__nv_bfloat16, 128, 0, false>(h, B, out) : plan_fma_t<float, 128, 0, false>(h, B, out);
    }
    if (h->cfg.d_v == 64)
        return bf ? plan_fma_t<__nv_bfloat16, 64, 16, GQA>(h, B, out) : plan_fma_t<float, 64, 16, GQA>(h, B, out);
    return bf ? plan_fma_t<__nv_bfloat16, 128, 32, GQA>(h, B, out) : plan_fma_t<float, 128, 32, GQA>(h, B, out);
}

// Workspace: header ints, then partial outputs, then (max, sum) pairs.
struct WorkspaceLayout {
    size_t hdr_bytes, rec_o_bytes, rec_ml_bytes, total;
    int n_rec, sync_ints;
};

// Thread blocks the balanced partition launches at most, per kernel family; the workspace is sized from the same numbers
// the launchers use.
int mma_grid_cap(const gva_handle *h, bool gqa) {
#ifdef GVA_WITH_MMA
    if (h->cfg.cache_dtype == GVA_E4M3) return fp8_blocks_per_sm(h->cfg) * h->sm_count;
    return mma_blocks_per_sm_cap(h->cfg, gqa, h->smem_per_sm) * h->sm_count;
#else
    (void)gqa;
    return 0;
#endif
}
int fma_grid_cap(const gva_handle *h) { return 4 * h->sm_count; }

// Upper bound on units of the balanced partition (records per sequence come on top): the CUDA-core kernel uses one unit
// per block; the tensor-core kernels cut every range into a head and, for d_v = 64, GVA_TAIL_UNITS tails.
int max_units_balanced(const gva_handle *h) {
    int units = 0;
#ifdef GVA_WITH_MMA
    const int per_range = h->cfg.d_v == 64 ? GVA_TAIL_UNITS + 1 : 1;
    const int cap = std::max(mma_grid_cap(h, false), mma_grid_cap(h, true));
    units = cap * per_range;
    const bool fma_possible = h->cfg.cache_dtype == GVA_F32 || h->cfg.kernel == GVA_KERNEL_FMA ||
                              (h->cfg.cache_dtype == GVA_BF16 && !(mma_supported(h->cfg, false) && mma_supported(h->cfg, true)));
#else
    const bool fma_possible = true;
#endif
    if (fma_possible) units = std::max(units, fma_grid_cap(h));
    return units;
}
int max_rec_mult(const gva_handle *h) {
#ifdef GVA_WITH_MMA
    if (h->cfg.cache_dtype == GVA_E4M3) return GVA_FP8_WPG;
    return h->cfg.d_v == 64 ? GVA_MMA_WPG64 : 1;
#else
    return 1;
#endif
}

WorkspaceLayout workspace_layout(const gva_handle *h, int B, int num_splits, int q_len = 1) {
    WorkspaceLayout w;
    w.n_rec = max_rec_mult(h) * (num_splits > 0 ? B * num_splits : max_units_balanced(h) + B);
    if (w.n_rec < 1) w.n_rec = 1;
    const size_t HQ = (size_t)h->cfg.H * q_len;             // q_len * H pseudo-heads per record
    w.hdr_bytes = align_up((size_t)(kHdrInts + 2 * B) * 4, 256);
    w.rec_o_bytes = align_up((size_t)w.n_rec * HQ * h->cfg.d_v * 4, 256);
    w.rec_ml_bytes = align_up((size_t)w.n_rec * HQ * 2 * 4, 256);
    w.total = w.hdr_bytes + w.rec_o_bytes + w.rec_ml_bytes;
    w.sync_ints = kSyncWords;
    return w;
}

int check_common(const gva_handle *h, int B, int max_seq_len, int num_splits) {
    if (!h) return GVA_ERR_INVALID_ARG;
    if (B < 0 || max_seq_len < 0 || num_splits < 0) return GVA_ERR_INVALID_ARG;
    if (B > 8192 || num_splits > 4096) return GVA_ERR_UNSUPPORTED;
    // total tiles must fit an int with headroom
    if ((long long)B * ((max_seq_len + 31) / 32 + 1) >= (1ll << 30)) return GVA_ERR_UNSUPPORTED;
    return GVA_OK;
}

// Validates and launches one decode kernel (which also merges its partial results).  dry = true runs every host-side
// check and preparation (workspace, kernel choice, shared-memory fit, tensor maps, sync region) but launches nothing, so
// that a caller can make sure a later launch cannot fail for a reason known in advance.
template <bool GQA>
int launch_decode(gva_handle *h, DecodeParams p, void *workspace, size_t workspace_bytes, int B, int max_seq_len,
                  int num_splits, cudaStream_t stream, int q_len = 1, bool dry = false) {
    const WorkspaceLayout w = workspace_layout(h, B, num_splits, q_len);
    if (!workspace || workspace_bytes < w.total) return GVA_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return GVA_ERR_INVALID_ARG;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    p.hdr = reinterpret_cast<int32_t *>(ws);
    p.rec_o = reinterpret_cast<float *>(ws + w.hdr_bytes);
    p.rec_ml = reinterpret_cast<float *>(ws + w.hdr_bytes + w.rec_o_bytes);
    p.n_rec = w.n_rec;
    p.num_splits = num_splits;
    p.rec_mult = 1;
    if (B == 0) return GVA_OK;

    int kernel = h->cfg.kernel;
    if (kernel == GVA_KERNEL_AUTO) {
#ifdef GVA_WITH_MMA
        kernel = (h->cfg.cache_dtype == GVA_BF16 && mma_supported(h->cfg, GQA)) ? GVA_KERNEL_MMA : GVA_KERNEL_FMA;
#else
        kernel = GVA_KERNEL_FMA;
#endif
    }
    if (h->cfg.cache_dtype == GVA_E4M3) kernel = GVA_KERNEL_MMA;
    if (q_len > 1 && (GQA || kernel != GVA_KERNEL_MMA)) return GVA_ERR_UNSUPPORTED;   // multi-token decode: tensor-core kernel only
    const int rc_sync = ensure_sync(h, w.sync_ints, stream);
    if (rc_sync != GVA_OK) return rc_sync;
    p.sync = h->sync_base + h->sync_off;
    p.epoch = dry ? h->epoch : ++h->epoch;      // a dry run prepares, it does not consume an epoch
    p.hdr_stamp = (int)((((unsigned)h->serial & 2047u) << 20) | ((unsigned)p.epoch & 0xfffffu)) + 1;
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) {
            (void)cudaGetLastError();
            cap = cudaStreamCaptureStatusActive;      // cannot tell: take the safe side
        }
        if (cap != cudaStreamCaptureStatusNone) p.hdr_stamp = 0;
    }
    if (h->epoch >= (1 << 30)) h->epoch = 2 + (h->epoch & 1);      // wrap, keeping the parity sequence
    if (kernel == GVA_KERNEL_MMA) {
#ifdef GVA_WITH_MMA
        h->mma.dry = dry;
        int rc = h->cfg.cache_dtype == GVA_E4M3
                     ? launch_decode_fp8(h->cfg, h->mma, h->sm_count, h->smem_optin, p, B, q_len, max_seq_len, num_splits, stream,
                                         &h->last_num_splits, &h->last_tile, &p.rec_mult, GQA)
                 : q_len > 1 ? launch_decode_mma_multi(h->cfg, h->mma, h->sm_count, h->smem_optin, p, B, q_len, max_seq_len, num_splits,
                                                     mma_grid_cap(h, false), stream, &h->last_num_splits, &h->last_tile, &p.rec_mult)
                           : launch_decode_mma<GQA>(h->cfg, h->mma, h->sm_count, h->smem_optin, p, B, max_seq_len, num_splits,
                                        mma_grid_cap(h, GQA), stream, &h->last_num_splits, &h->last_tile, &p.rec_mult);
        h->mma.dry = false;
        if (rc != GVA_OK) return rc;
        h->last_kernel = GVA_KERNEL_MMA;
#else
        return GVA_ERR_UNSUPPORTED;
#endif
    } else {
        FmaPlan plan;
        if (!plan_fma<GQA>(h, B, &plan)) return GVA_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(plan.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem) != cudaSuccess)
            return GVA_ERR_CUDA;
        int grid;
        if (num_splits > 0) {
            grid = B * num_splits;
        } else {
            int per_sm = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, plan.fn, plan.threads, plan.smem) != cudaSuccess)
                return GVA_ERR_CUDA;
            if (per_sm < 1) per_sm = 1;
            const long long tiles_ub = (long long)B * ((max_seq_len + 31) / 32);
            grid = (int)std::min<long long>(std::min<long long>((long long)per_sm * h->sm_count, fma_grid_cap(h)),
                                            std::max<long long>(tiles_ub, 1));
        }
        h->last_num_splits = grid;
        h->last_kernel = GVA_KERNEL_FMA;
        h->last_tile = 32;
        if (dry) return GVA_OK;
        if (launch_pdl(plan.fn, dim3(grid), dim3(plan.threads), plan.smem, stream, p) != cudaSuccess) {
            (void)cudaGetLastError();
            return GVA_ERR_CUDA;
        }
    }
    if (dry) return GVA_OK;
    // Warps per head for the merge: enough that a head's records (about units / B, plus the cuts at both ends)
    // are fetched in one or two round trips; one warp per head and four heads per block for the wide-head shape
    // unless a sequence has many records, so that those blocks fit beside the decode kernel's blocks.
    const long long tiles_ub = (long long)B * ((max_seq_len + h->last_tile - 1) / h->last_tile);
    const UnitPlan est = make_unit_plan((int)tiles_ub, h->last_num_splits,
                                        h->cfg.d_v == 64 && h->last_kernel == GVA_KERNEL_MMA);
    const int units = num_splits > 0 ? num_splits : plan_units(est);
    const int n_est = (num_splits > 0 ? units : units / B + 8) * p.rec_mult;
    int wph = h->cfg.d_v == 64 ? 4 : 1;
    while (wph < 32 && wph * 8 < n_est) wph *= 2;
    if (h->cfg.d_v == 128 && wph <= 2) wph = 1;
    // ... but no more warps in the whole grid than fit beside the decode blocks (64 registers per merge thread next to
    // two 160-thread decode blocks of ~72 registers: about 27 warps per SM at the 48 registers of the small instantiation): merge blocks that are not resident start
    // only when decode blocks leave, a launch latency after the last tile instead of a poll after it
    // (measured on the 32-sequence long-context workload: the last poll succeeds 2.7 us after the last arrival when
    // part of the merge grid is not resident, 1.4 us when all of it is)
    const int HQ = h->cfg.H * q_len;           // the merge sees q_len * H pseudo-heads: out rows are [b][slot][head]
    p.H = HQ;
    while (wph > 1 && (long long)B * HQ * wph > 4096) wph /= 2;
    const int hpb = wph >= 4 ? 1 : 4 / wph;
    const size_t csmem = (size_t)wph * hpb * (h->cfg.d_v + 2) * sizeof(float);
    const dim3 cgrid(B, (HQ + hpb - 1) / hpb), cblock(32 * wph * hpb);
    const cudaError_t ce = (h->cfg.d_v == 64) ? launch_pdl(combine_kernel<64>, cgrid, cblock, csmem, stream, p, wph, hpb)
                                              : launch_pdl(combine_kernel<128>, cgrid, cblock, csmem, stream, p, wph, hpb);
    if (ce != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

}  // namespace

extern "C" {

int gva_create(gva_handle **out, const gva_config *cfg, int device) {
    if (!out || !cfg) return GVA_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->H <= 0 || cfg->G <= 0 || cfg->d_v <= 0 || cfg->d_c <= 0 || cfg->d_r < 0 || cfg->page_size <= 0 ||
        !(cfg->rope_base > 1.0) || !(cfg->softmax_scale >= 0.f) || device < 0)
        return GVA_ERR_INVALID_ARG;
    if (cfg->cache_dtype != GVA_F32 && cfg->cache_dtype != GVA_BF16 && cfg->cache_dtype != GVA_E4M3) return GVA_ERR_INVALID_ARG;
    if (cfg->kernel < GVA_KERNEL_AUTO || cfg->kernel > GVA_KERNEL_MMA) return GVA_ERR_INVALID_ARG;
    if (cfg->H % cfg->G != 0 || cfg->H / cfg->G != kHeadsPerGroup) return GVA_ERR_UNSUPPORTED;
    // d_r = 0 is the value-only cache (no positional slice: half the bytes of matched GQA, Section 3.4)
    if (!((cfg->d_v == 64 && (cfg->d_r == 16 || cfg->d_r == 24 || cfg->d_r == 0)) || (cfg->d_v == 128 && (cfg->d_r == 32 || cfg->d_r == 0))))
        return GVA_ERR_UNSUPPORTED;
    if (cfg->G > 8 || cfg->d_c > 256 || cfg->page_size % 32 != 0) return GVA_ERR_UNSUPPORTED;
    if (cfg->kernel == GVA_KERNEL_MMA && cfg->cache_dtype == GVA_F32) return GVA_ERR_UNSUPPORTED;
    if (cfg->cache_dtype == GVA_E4M3) {   // the 8-bit cache: one shape, tensor-core kernel only
#ifdef GVA_WITH_MMA
        if (cfg->kernel == GVA_KERNEL_FMA || !fp8_supported(*cfg)) return GVA_ERR_UNSUPPORTED;
#else
        return GVA_ERR_UNSUPPORTED;
#endif
    }
#ifndef GVA_WITH_MMA
    if (cfg->kernel == GVA_KERNEL_MMA) return GVA_ERR_UNSUPPORTED;
#endif

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) return GVA_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return GVA_ERR_CUDA;
    int major = 0, sms = 0, optin = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, device) != cudaSuccess)
        return GVA_ERR_CUDA;
    if (major != 10) return GVA_ERR_CUDA;   // the kernels are built for sm_100a only

    gva_handle *h = new (std::nothrow) gva_handle();
    if (!h) return GVA_ERR_INVALID_ARG;
    h->cfg = *cfg;
    h->device = device;
    h->sm_count = sms;
    h->smem_optin = optin;
    h->smem_per_sm = per_sm;
    h->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : (float)(1.0 / std::sqrt((double)(cfg->d_c + cfg->d_r)));
    for (int i = 0; i < kMaxRopePairs; ++i)
        h->rope.inv_freq[i] = (2 * i < cfg->d_r) ? std::pow(cfg->rope_base, -2.0 * (double)i / (double)cfg->d_r) : 0.0;
    h->last_num_splits = 0;
    h->last_kernel = 0;
    h->last_tile = 0;
    {
        void *base = nullptr;
        if (cudaGetSymbolAddress(&base, g_sync_arena) != cudaSuccess) {     // `device` is current
            (void)cudaGetLastError();
            delete h;
            return GVA_ERR_CUDA;
        }
        h->sync_base = static_cast<int32_t *>(base);
        h->sync_off = h->sync_cap = h->n_regions = 0;
        h->epoch = 0;
        static std::atomic<int> n_handles{0};
        h->serial = n_handles.fetch_add(1);
    }
#ifdef GVA_WITH_MMA
    int rc = mma_host_init(&h->mma, device);
    if (rc != GVA_OK) {
        delete h;
        return rc;
    }
#endif
    // the absorb kernel may need more than 48 KB for a 128 x 128 map
    const size_t absorb_smem = absorb_smem_bytes(cfg->d_v, cfg->d_c);
    if (absorb_smem > (size_t)optin ||
        cudaFuncSetAttribute(absorb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)absorb_smem) != cudaSuccess ||
        cudaFuncSetAttribute(step_front_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)absorb_smem) != cudaSuccess ||
        cudaFuncSetAttribute(step_front_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)absorb_smem) !=
            cudaSuccess ||
        cudaFuncSetAttribute(step_front_kernel<uint8_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)absorb_smem) !=
            cudaSuccess) {
        delete h;
        return GVA_ERR_CUDA;
    }
    *out = h;
    return GVA_OK;
}

int gva_destroy(gva_handle *h) {
    if (!h) return GVA_ERR_INVALID_ARG;
    for (int i = 0; i < h->n_regions; ++i) arena_release(h->region_off[i], h->region_cap[i]);
    delete h;
    return GVA_OK;
}

size_t gva_decode_workspace_bytes(const gva_handle *h, int B, int max_seq_len, int num_splits) {
    if (check_common(h, B, max_seq_len, num_splits) != GVA_OK) return 0;
    return workspace_layout(h, B, num_splits).total;
}

int gva_absorb_query(gva_handle *h, const float *q_c, const float *q_r, const float *M, const int32_t *q_pos,
                     float *q_abs, int B, void *stream) {
    if (!h || B < 0) return GVA_ERR_INVALID_ARG;
    if (B == 0) return GVA_OK;
    if (!q_c || (h->cfg.d_r > 0 && !q_r) || !M || !q_pos || !q_abs) return GVA_ERR_INVALID_ARG;
    if (!aligned(q_c, 4) || !aligned(q_r, 4) || !aligned(M, 4) || !aligned(q_pos, 4) || !aligned(q_abs, 16))
        return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    const size_t smem = absorb_smem_bytes(c.d_v, c.d_c);
    // many rows (prefill): a batch of small GEMMs on the tensor cores (f16 hi/lo operands, f32-level accuracy)
    const bool vec_ok = aligned(q_c, 16) && aligned(M, 16) && aligned(q_r, 8);
    if (B >= 512 && vec_ok && ((c.d_v == 64 && c.d_c == 64) || (c.d_v == 128 && c.d_c == 128))) {
        const int chunk = kAbsorbMmaRows;
        const size_t smem_mma = c.d_v == 64 ? AbsorbMmaTraits<64, 64>::smem_bytes() : AbsorbMmaTraits<128, 128>::smem_bytes();
        int per_head = (4 * h->sm_count + c.H - 1) / c.H;                 // about four blocks per SM in all
        int rows_per_block = (B + per_head - 1) / per_head;
        rows_per_block = (rows_per_block + chunk - 1) / chunk * chunk;
        const dim3 g2(c.H, (B + rows_per_block - 1) / rows_per_block);
        auto fn = c.d_v == 64 ? absorb_rows_mma_kernel<64, 64> : absorb_rows_mma_kernel<128, 128>;
        if (smem_mma > (size_t)h->smem_optin ||
            cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_mma) != cudaSuccess)
            return GVA_ERR_CUDA;
        if (launch_pdl(fn, g2, dim3(kAbsorbMmaThreads), smem_mma, static_cast<cudaStream_t>(stream), q_c, q_r, M, q_pos, q_abs,
                       B, c.H, c.d_r, rows_per_block, h->rope) != cudaSuccess) {
            (void)cudaGetLastError();
            return GVA_ERR_CUDA;
        }
        return GVA_OK;
    }
    dim3 grid(c.H, (B + kAbsorbBatch - 1) / kAbsorbBatch);
    if (launch_pdl(absorb_kernel, grid, dim3(kAbsorbThreads), smem, static_cast<cudaStream_t>(stream), q_c, q_r, M, q_pos,
                   q_abs, B, c.H, c.d_v, c.d_c, c.d_r, h->rope) != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

int gva_append_cache(gva_handle *h, const gva_cache *cache, const float *v_new, const float *kr_new,
                     const int32_t *pos, int B, int32_t *dev_status, void *stream) {
    if (!h || !cache || B < 0) return GVA_ERR_INVALID_ARG;
    if (B == 0) return GVA_OK;
    if (!cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool) || !v_new || (h->cfg.d_r > 0 && !kr_new) || !pos) return GVA_ERR_INVALID_ARG;
    if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
    if (!aligned(cache->v_pool, 16) || !aligned(cache->kr_pool, 16)) return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c.G * c.d_v > kAppendMaxPerThread * 128) return GVA_ERR_UNSUPPORTED;
    cudaError_t ce;
    if (c.cache_dtype == GVA_E4M3)
        ce = launch_pdl(append_kernel<uint8_t>, dim3(B), dim3(128), 0, s, static_cast<uint8_t *>(cache->v_pool),
                        static_cast<uint8_t *>(cache->kr_pool), cache->block_table, v_new, kr_new, pos, c.G, c.d_v,
                        c.d_r, c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope);
    else if (c.cache_dtype == GVA_BF16)
        ce = launch_pdl(append_kernel<__nv_bfloat16>, dim3(B), dim3(128), 0, s, static_cast<__nv_bfloat16 *>(cache->v_pool),
                        static_cast<__nv_bfloat16 *>(cache->kr_pool), cache->block_table, v_new, kr_new, pos, c.G, c.d_v,
                        c.d_r, c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope);
    else
        ce = launch_pdl(append_kernel<float>, dim3(B), dim3(128), 0, s, static_cast<float *>(cache->v_pool),
                        static_cast<float *>(cache->kr_pool), cache->block_table, v_new, kr_new, pos, c.G, c.d_v, c.d_r,
                        c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope);
    if (ce != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

int gva_append_chunk(gva_handle *h, const gva_cache *cache, const float *v_new, const float *kr_new, const int32_t *cu_q,
                     const int32_t *ctx_lens, int B, int n_q, int32_t *dev_status, void *stream) {
    if (!h || !cache || B < 0 || n_q < 0) return GVA_ERR_INVALID_ARG;
    if (B == 0 || n_q == 0) return GVA_OK;
    if (!cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool) || !v_new || (h->cfg.d_r > 0 && !kr_new) || !cu_q || !ctx_lens) return GVA_ERR_INVALID_ARG;
    if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
    if (!aligned(cache->v_pool, 16) || !aligned(cache->kr_pool, 16)) return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c.G * c.d_v > kAppendMaxPerThread * 128) return GVA_ERR_UNSUPPORTED;
    const int vec4 = (aligned(v_new, 16) && (c.G * c.d_v) % 4 == 0) ? 1 : 0;
    cudaError_t ce;
    if (c.cache_dtype == GVA_E4M3)
        ce = launch_pdl(append_chunk_kernel<uint8_t>, dim3((n_q + kAppendChunkRows - 1) / kAppendChunkRows), dim3(128), 0, s, static_cast<uint8_t *>(cache->v_pool),
                        static_cast<uint8_t *>(cache->kr_pool), cache->block_table, v_new, kr_new, cu_q, ctx_lens, B, c.G,
                        c.d_v, c.d_r, c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope, vec4);
    else if (c.cache_dtype == GVA_BF16)
        ce = launch_pdl(append_chunk_kernel<__nv_bfloat16>, dim3((n_q + kAppendChunkRows - 1) / kAppendChunkRows), dim3(128), 0, s, static_cast<__nv_bfloat16 *>(cache->v_pool),
                        static_cast<__nv_bfloat16 *>(cache->kr_pool), cache->block_table, v_new, kr_new, cu_q, ctx_lens, B, c.G,
                        c.d_v, c.d_r, c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope, vec4);
    else
        ce = launch_pdl(append_chunk_kernel<float>, dim3((n_q + kAppendChunkRows - 1) / kAppendChunkRows), dim3(128), 0, s, static_cast<float *>(cache->v_pool),
                        static_cast<float *>(cache->kr_pool), cache->block_table, v_new, kr_new, cu_q, ctx_lens, B, c.G, c.d_v,
                        c.d_r, c.page_size, cache->num_pages, cache->max_pages_per_seq, dev_status, h->rope, vec4);
    if (ce != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}

static int prefill_impl(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q, const int32_t *ctx_lens,
                        float *out, float *lse, void *workspace, size_t workspace_bytes, int B, int n_q, int max_q_len,
                        int num_splits, int32_t *dev_status, void *stream) {
    if (!h || !cache || B < 0 || max_q_len < 0 || n_q < 0 || num_splits < 1) return GVA_ERR_INVALID_ARG;
    if (B == 0 || max_q_len == 0) return GVA_OK;
    if (!cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool) || !q_abs || !cu_q || !ctx_lens || !out) return GVA_ERR_INVALID_ARG;
    if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
    if (!aligned(cache->v_pool, 16) || !aligned(cache->kr_pool, 16) || !aligned(q_abs, 16) || !aligned(out, 16))
        return GVA_ERR_INVALID_ARG;
    if (B > 65535) return GVA_ERR_UNSUPPORTED;
#ifdef GVA_WITH_MMA
    const gva_config &c = h->cfg;
    PrefillParams p;
    std::memset(&p, 0, sizeof(p));
    p.q_abs = q_abs;
    p.cu_q = cu_q;
    p.ctx_lens = ctx_lens;
    p.block_table = cache->block_table;
    p.out = out;
    p.lse = lse;
    p.dev_status = dev_status;
    p.B = B;
    p.H = c.H;
    p.G = c.G;
    p.P = c.page_size;
    p.num_pages = cache->num_pages;
    p.max_pages = cache->max_pages_per_seq;
    p.scale_log2 = h->scale * kLog2e;
    p.num_splits = num_splits;
    if (num_splits > 1) {
        const size_t o_bytes = align_up((size_t)n_q * c.H * num_splits * c.d_v * sizeof(float), 256);
        const size_t ml_bytes = (size_t)n_q * c.H * num_splits * 2 * sizeof(float);
        if (!workspace || !aligned(workspace, 256) || workspace_bytes < o_bytes + ml_bytes) return GVA_ERR_WORKSPACE;
        p.part_o = static_cast<float *>(workspace);
        p.part_ml = reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + o_bytes);
    }
    return launch_prefill(c, h->mma, h->smem_optin, p, cache->v_pool, cache->kr_pool, B, max_q_len, n_q,
                          static_cast<cudaStream_t>(stream));
#else
    return GVA_ERR_UNSUPPORTED;
#endif
}

int gva_prefill(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q, const int32_t *ctx_lens,
                float *out, float *lse, int B, int max_q_len, int32_t *dev_status, void *stream) {
    return prefill_impl(h, cache, q_abs, cu_q, ctx_lens, out, lse, nullptr, 0, B, 0, max_q_len, 1, dev_status, stream);
}

// Splits per query block for gva_decode_multi.  Automatic choice: the split count that minimises
// (waves of thread blocks over the 2-per-SM slots) x (tiles per block + a fixed per-block cost of about 6 tiles),
// so that the last wave is not left mostly empty; never more splits than tiles, at most 64.
static int multi_splits(const gva_handle *h, int B, int max_q_len, int max_seq_len, int num_splits) {
    const int tiles = (max_seq_len + 63) / 64;
    int s = num_splits;
    if (s <= 0) {
        const long long blocks = (long long)B * h->cfg.G * ((max_q_len + 31) / 32);
        const long long slots = 2LL * h->sm_count;
        long long best = -1;
        s = 1;
        for (int c = 1; c <= 64 && c <= (tiles > 0 ? tiles : 1); ++c) {
            const long long waves = (blocks * c + slots - 1) / slots;
            const long long cost = waves * ((tiles + c - 1) / c + 6);
            if (best < 0 || cost < best) {
                best = cost;
                s = c;
            }
        }
    }
    if (s > tiles) s = tiles;
    if (s > 64) s = 64;
    return s < 1 ? 1 : s;
}

size_t gva_decode_multi_workspace_bytes(const gva_handle *h, int B, int n_q, int max_q_len, int max_seq_len, int num_splits) {
    if (!h || B < 0 || n_q < 0 || max_q_len < 0 || max_seq_len < 0) return 0;
    const int s = multi_splits(h, B, max_q_len, max_seq_len, num_splits);
    if (s == 1) return 256;
    return align_up((size_t)n_q * h->cfg.H * s * h->cfg.d_v * sizeof(float), 256) +
           align_up((size_t)n_q * h->cfg.H * s * 2 * sizeof(float), 256);
}

int gva_decode_multi(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q, const int32_t *ctx_lens,
                     float *out, float *lse, void *workspace, size_t workspace_bytes, int B, int n_q, int max_q_len,
                     int max_seq_len, int num_splits, int32_t *dev_status, void *stream) {
    if (!h || max_seq_len < 0 || num_splits < 0) return GVA_ERR_INVALID_ARG;
    const int s = multi_splits(h, B > 0 ? B : 1, max_q_len, max_seq_len, num_splits);
    return prefill_impl(h, cache, q_abs, cu_q, ctx_lens, out, lse, workspace, workspace_bytes, B, n_q, max_q_len, s, dev_status,
                        stream);
}

static int decode_impl(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens, float *out,
                       float *lse, void *workspace, size_t workspace_bytes, int B, int max_seq_len, int num_splits,
                       int32_t *dev_status, void *stream, int early_start, const int32_t *append_pos, int q_len = 1,
                       bool dry = false, const int32_t *cu_q = nullptr) {
    int rc = check_common(h, B, max_seq_len, num_splits);
    if (rc != GVA_OK) return rc;
    if (!cache) return GVA_ERR_INVALID_ARG;
    if (B > 0) {
        if (!cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool) || !q_abs || !seq_lens || !out) return GVA_ERR_INVALID_ARG;
        if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
        if (!aligned(cache->v_pool, 16) || !aligned(cache->kr_pool, 16) || !aligned(q_abs, 16) || !aligned(out, 16))
            return GVA_ERR_INVALID_ARG;
    }
    const gva_config &c = h->cfg;
    DecodeParams p;
    std::memset(&p, 0, sizeof(p));
    p.v_pool = cache->v_pool;
    p.kr_pool = cache->kr_pool;
    p.block_table = cache->block_table;
    p.seq_lens = seq_lens;
    p.q = q_abs;
    p.out = out;
    p.lse = lse;
    p.dev_status = dev_status;
    p.B = B; p.H = c.H; p.G = c.G; p.P = c.page_size;
    p.num_pages = cache->num_pages;
    p.max_pages = cache->max_pages_per_seq;
    p.scale_log2 = h->scale * kLog2e;
    p.early_start = early_start;
    p.append_pos = append_pos;
    p.q_len = q_len;
    p.cu_q = cu_q;
    return launch_decode<false>(h, p, workspace, workspace_bytes, B, max_seq_len, num_splits,
                                static_cast<cudaStream_t>(stream), q_len, dry);
}

int gva_decode(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens, float *out,
               float *lse, void *workspace, size_t workspace_bytes, int B, int max_seq_len, int num_splits,
               int32_t *dev_status, void *stream) {
    return decode_impl(h, cache, q_abs, seq_lens, out, lse, workspace, workspace_bytes, B, max_seq_len, num_splits,
                       dev_status, stream, 0, nullptr);
}

size_t gva_decode_tokens_workspace_bytes(const gva_handle *h, int B, int q_len, int max_seq_len, int num_splits) {
    if (check_common(h, B, max_seq_len, num_splits) != GVA_OK || q_len < 2 || q_len > 8) return 0;
    return workspace_layout(h, B, num_splits, q_len).total;
}

int gva_decode_tokens(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens, float *out, float *lse,
                      void *workspace, size_t workspace_bytes, int B, int q_len, int max_seq_len, int num_splits,
                      int32_t *dev_status, void *stream) {
    if (!h) return GVA_ERR_INVALID_ARG;
    if (q_len < 2 || q_len > 8) return GVA_ERR_UNSUPPORTED;
    return decode_impl(h, cache, q_abs, seq_lens, out, lse, workspace, workspace_bytes, B, max_seq_len, num_splits, dev_status,
                       stream, 0, nullptr, q_len);
}

int gva_decode_tokens_ragged(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q, const int32_t *seq_lens,
                             float *out, float *lse, void *workspace, size_t workspace_bytes, int B, int max_q_len, int max_seq_len,
                             int num_splits, int32_t *dev_status, void *stream) {
    if (!h || !cu_q) return GVA_ERR_INVALID_ARG;
    if (max_q_len < 1 || max_q_len > 8) return GVA_ERR_UNSUPPORTED;
    return decode_impl(h, cache, q_abs, seq_lens, out, lse, workspace, workspace_bytes, B, max_seq_len, num_splits, dev_status,
                       stream, 0, nullptr, max_q_len < 2 ? 2 : max_q_len, false, cu_q);
}

int gva_decode_step(gva_handle *h, const gva_cache *cache, const float *M, const float *q_c, const float *q_r,
                    const float *v_new, const float *kr_new, const int32_t *pos, const int32_t *seq_lens, float *q_abs,
                    float *out, float *lse, void *workspace, size_t workspace_bytes, int B, int max_seq_len,
                    int num_splits, int32_t *dev_status, void *stream) {
    int rc = check_common(h, B, max_seq_len, num_splits);
    if (rc != GVA_OK) return rc;
    if (B == 0) return GVA_OK;
    if (!cache || !M || !q_c || (h->cfg.d_r > 0 && !q_r) || !v_new || (h->cfg.d_r > 0 && !kr_new) || !pos || !seq_lens || !q_abs || !out)
        return GVA_ERR_INVALID_ARG;
    if (!cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool) || cache->num_pages <= 0 || cache->max_pages_per_seq <= 0)
        return GVA_ERR_INVALID_ARG;
    if (!aligned(cache->v_pool, 16) || !aligned(cache->kr_pool, 16) || !aligned(q_abs, 16) || !aligned(out, 16) ||
        !aligned(M, 16))
        return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    if (c.G * c.d_v > kAppendMaxPerThread * 128) return GVA_ERR_UNSUPPORTED;
    // every host-side check of the decode launch comes first, so that an error return means nothing was enqueued and
    // the cache was not advanced
#ifndef GVA_NO_DRY
    rc = decode_impl(h, cache, q_abs, seq_lens, out, lse, workspace, workspace_bytes, B, max_seq_len, num_splits, dev_status,
                     stream, 1, pos, 1, true);
    if (rc != GVA_OK) return rc;
#endif
    StepFrontParams a;
    a.q_c = q_c; a.q_r = q_r; a.M = M; a.v_new = v_new; a.kr_new = kr_new;
    a.pos = pos; a.block_table = cache->block_table; a.q_abs = q_abs;
    a.v_pool = cache->v_pool; a.kr_pool = cache->kr_pool; a.dev_status = dev_status;
    a.B = B; a.H = c.H; a.G = c.G; a.d_v = c.d_v; a.d_c = c.d_c; a.d_r = c.d_r; a.P = c.page_size;
    a.num_pages = cache->num_pages; a.max_pages = cache->max_pages_per_seq;
    // sequences per absorb item: 16 where that keeps the grid at one block per SM and the thread mapping allows it
    a.fold = c.H * ((B + kAbsorbBatch - 1) / kAbsorbBatch) + B > h->sm_count ? 1 : 0;
    a.batch = (a.fold && kAbsorbBatchMax * c.d_v <= 4 * kAbsorbThreads) ? kAbsorbBatchMax : kAbsorbBatch;
    a.n_absorb = c.H * ((B + a.batch - 1) / a.batch);
    const int front_grid = a.fold ? (a.n_absorb > B ? a.n_absorb : B) : a.n_absorb + B;
    a.trace_call = h->epoch + 1;
    const size_t smem = absorb_smem_bytes(c.d_v, c.d_c);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const cudaError_t ce = (c.cache_dtype == GVA_E4M3)
        ? launch_pdl(step_front_kernel<uint8_t>, dim3(front_grid), dim3(kAbsorbThreads), smem, st, a, h->rope)
        : (c.cache_dtype == GVA_BF16)
        ? launch_pdl(step_front_kernel<__nv_bfloat16>, dim3(front_grid), dim3(kAbsorbThreads), smem, st, a, h->rope)
        : launch_pdl(step_front_kernel<float>, dim3(front_grid), dim3(kAbsorbThreads), smem, st, a, h->rope);
    if (ce != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return decode_impl(h, cache, q_abs, seq_lens, out, lse, workspace, workspace_bytes, B, max_seq_len, num_splits,
                       dev_status, stream, 1, pos);
}

// ---- gva_decode without caller scratch ---------------------------------------------------------
// The split-KV partial results of gva_decode_static live in this array.  In host code the name is
// only a stand-in for the symbol; the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[GVA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on `device` (which must be current); nullptr on failure.
void *static_scratch_for(int device) {
    if (device < 0 || device >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_static_ptr[device] = ptr;
    }
    return g_static_ptr[device];
}
}  // namespace

int gva_decode_static(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens, float *out,
                      float *lse, int B, int max_seq_len, int num_splits, int32_t *dev_status, void *stream) {
    int rc = check_common(h, B, max_seq_len, num_splits);
    if (rc != GVA_OK) return rc;
    if (workspace_layout(h, B, num_splits).total > (size_t)GVA_STATIC_SCRATCH_BYTES) return GVA_ERR_STATIC_LIMIT;
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess) return GVA_ERR_CUDA;
    if (current != h->device) return GVA_ERR_INVALID_ARG;
    void *scratch = static_scratch_for(current);
    if (!scratch) return GVA_ERR_CUDA;
    return gva_decode(h, cache, q_abs, seq_lens, out, lse, scratch, (size_t)GVA_STATIC_SCRATCH_BYTES, B, max_seq_len,
                      num_splits, dev_status, stream);
}

int gqa_decode(gva_handle *h, const gqa_cache *cache, const float *q, const int32_t *seq_lens, float *out, float *lse,
               void *workspace, size_t workspace_bytes, int B, int max_seq_len, int num_splits, int32_t *dev_status,
               void *stream) {
    int rc = check_common(h, B, max_seq_len, num_splits);
    if (rc != GVA_OK) return rc;
    if (!cache) return GVA_ERR_INVALID_ARG;
    if (B > 0) {
        if (!cache->k_pool || !cache->v_pool || !q || !seq_lens || !out) return GVA_ERR_INVALID_ARG;
        if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
        if (!aligned(cache->k_pool, 16) || !aligned(cache->v_pool, 16) || !aligned(q, 16) || !aligned(out, 16))
            return GVA_ERR_INVALID_ARG;
    }
    const gva_config &c = h->cfg;
    DecodeParams p;
    std::memset(&p, 0, sizeof(p));
    p.v_pool = cache->v_pool;
    p.k_pool = cache->k_pool;
    p.block_table = cache->block_table;
    p.seq_lens = seq_lens;
    p.q = q;
    p.out = out;
    p.lse = lse;
    p.dev_status = dev_status;
    p.B = B; p.H = c.H; p.G = c.G; p.P = c.page_size;
    p.num_pages = cache->num_pages;
    p.max_pages = cache->max_pages_per_seq;
    p.scale_log2 = (float)(1.0 / std::sqrt((double)c.d_v)) * kLog2e;
    return launch_decode<true>(h, p, workspace, workspace_bytes, B, max_seq_len, num_splits,
                               static_cast<cudaStream_t>(stream));
}

namespace {
struct StepLayout {
    size_t q_c, q_r, v_new, kr_new, pos, lens, q_abs, out, ws, total, ws_bytes;
};
StepLayout step_layout(const gva_handle *h, int B, int num_splits) {
    const gva_config &c = h->cfg;
    StepLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
    L.q_c = take((size_t)B * c.H * c.d_c * 4);
    L.q_r = take((size_t)B * c.H * c.d_r * 4);
    L.v_new = take((size_t)B * c.G * c.d_v * 4);
    L.kr_new = take((size_t)B * c.d_r * 4);
    L.pos = take((size_t)B * 4);
    L.lens = take((size_t)B * 4);
    L.q_abs = take((size_t)B * c.H * (c.d_v + c.d_r) * 4);
    L.out = take((size_t)B * c.H * c.d_v * 4);
    L.ws_bytes = workspace_layout(h, B, num_splits).total;
    L.ws = take(L.ws_bytes);
    L.total = off;
    return L;
}
}  // namespace

size_t gva_step_scratch_bytes(const gva_handle *h, int B, int max_seq_len, int num_splits) {
    if (check_common(h, B, max_seq_len, num_splits) != GVA_OK) return 0;
    return step_layout(h, B, num_splits).total;
}

int gva_decode_step_host(gva_handle *h, const gva_cache *cache, const float *M, const float *q_c_host,
                         const float *q_r_host, const float *v_new_host, const float *kr_new_host,
                         const int32_t *pos_host, const int32_t *seq_lens_host, float *out_host, void *scratch,
                         size_t scratch_bytes, int B, int max_seq_len, int num_splits, int32_t *dev_status,
                         void *stream) {
    int rc = check_common(h, B, max_seq_len, num_splits);
    if (rc != GVA_OK) return rc;
    if (B == 0) return GVA_OK;
    const bool rope = h->cfg.d_r > 0;                    // a value-only cache has no positional inputs: q_r_host / kr_new_host may be NULL
    if (!cache || !M || !q_c_host || (rope && !q_r_host) || !v_new_host || (rope && !kr_new_host) || !pos_host || !seq_lens_host || !out_host)
        return GVA_ERR_INVALID_ARG;
    const StepLayout L = step_layout(h, B, num_splits);
    if (!scratch || scratch_bytes < L.total) return GVA_ERR_WORKSPACE;
    if (!aligned(scratch, 256)) return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    unsigned char *s = static_cast<unsigned char *>(scratch);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto h2d = [&](size_t off, const void *src, size_t bytes) {
        return cudaMemcpyAsync(s + off, src, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    };
    // Pinned (page-locked, device-mapped) host buffers are read and written by the kernels directly over the
    // interconnect: that replaces five small copies, each of which would cost a few microseconds of stream time,
    // by loads and stores inside kernels that run anyway.  Pageable buffers take the staged path.
    const void *hosts[5] = {q_c_host, q_r_host, v_new_host, kr_new_host, out_host};
    void *mapped[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool host_mapped = true;
    for (int i = 0; i < 5 && host_mapped; ++i) {
        if (!rope && (i == 1 || i == 3)) continue;      // unused inputs stay NULL
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, hosts[i]) != cudaSuccess) {
            (void)cudaGetLastError();
            host_mapped = false;
        } else if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) {
            host_mapped = false;
        } else {
            mapped[i] = attr.devicePointer;
        }
    }
    // positions and lengths go to device scratch (every decode block reads them): by one small kernel when they are
    // pinned, else by two copies
    {
        void *ints[2] = {nullptr, nullptr};
        const void *src[2] = {pos_host, seq_lens_host};
        bool ints_mapped = host_mapped;
        for (int i = 0; i < 2 && ints_mapped; ++i) {
            cudaPointerAttributes attr;
            if (cudaPointerGetAttributes(&attr, src[i]) != cudaSuccess) {
                (void)cudaGetLastError();
                ints_mapped = false;
            } else if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) {
                ints_mapped = false;
            } else {
                ints[i] = attr.devicePointer;
            }
        }
        if (ints_mapped) {
            if (launch_pdl(stage_ints_kernel, dim3(1), dim3(128), 0, st, static_cast<const int32_t *>(ints[0]),
                           static_cast<const int32_t *>(ints[1]), reinterpret_cast<int32_t *>(s + L.pos),
                           reinterpret_cast<int32_t *>(s + L.lens), B) != cudaSuccess) {
                (void)cudaGetLastError();
                return GVA_ERR_CUDA;
            }
        } else if (!h2d(L.pos, pos_host, (size_t)B * 4) || !h2d(L.lens, seq_lens_host, (size_t)B * 4)) {
            return GVA_ERR_CUDA;
        }
    }
    const int32_t *pos = reinterpret_cast<const int32_t *>(s + L.pos);
    const int32_t *lens = reinterpret_cast<const int32_t *>(s + L.lens);
    float *q_abs = reinterpret_cast<float *>(s + L.q_abs);
    if (host_mapped) {
        return gva_decode_step(h, cache, M, static_cast<const float *>(mapped[0]), static_cast<const float *>(mapped[1]),
                               static_cast<const float *>(mapped[2]), static_cast<const float *>(mapped[3]), pos, lens,
                               q_abs, static_cast<float *>(mapped[4]), nullptr, s + L.ws, L.ws_bytes, B, max_seq_len,
                               num_splits, dev_status, stream);
    }
    if (!h2d(L.q_c, q_c_host, (size_t)B * c.H * c.d_c * 4) || (rope && !h2d(L.q_r, q_r_host, (size_t)B * c.H * c.d_r * 4)) ||
        !h2d(L.v_new, v_new_host, (size_t)B * c.G * c.d_v * 4) || (rope && !h2d(L.kr_new, kr_new_host, (size_t)B * c.d_r * 4)))
        return GVA_ERR_CUDA;
    float *out = reinterpret_cast<float *>(s + L.out);
    rc = gva_decode_step(h, cache, M, reinterpret_cast<const float *>(s + L.q_c), rope ? reinterpret_cast<const float *>(s + L.q_r) : nullptr,
                         reinterpret_cast<const float *>(s + L.v_new), rope ? reinterpret_cast<const float *>(s + L.kr_new) : nullptr, pos,
                         lens, q_abs, out, nullptr, s + L.ws, L.ws_bytes, B, max_seq_len, num_splits, dev_status, stream);
    if (rc != GVA_OK) return rc;
    if (cudaMemcpyAsync(out_host, out, (size_t)B * c.H * c.d_v * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GVA_ERR_CUDA;
    return GVA_OK;
}

}  // extern "C"

// ---- projections around the attention -----------------------------------------------------------------
namespace {
// host: double -> bf16 bits, round to nearest even (via round-to-odd f32, as on the device)
uint16_t host_bf16_from_double(double x) {
    float f = (float)x;                                   // nearest-even
    if ((double)f != x && std::isfinite(f)) {            // make it round-to-odd: step toward x's side, then set the sticky bit
        uint32_t u;
        std::memcpy(&u, &f, 4);
        const bool over = std::fabs((double)f) > std::fabs(x);
        if (over) u -= 1;                                 // truncate toward zero (magnitude)
        u |= 1u;
        std::memcpy(&f, &u, 4);
    }
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

int input_width(const gva_config &c) { return c.H * (c.d_v + c.d_r) + c.G * c.d_v + c.d_r; }

template <int MODE>
int launch_project(const gva_handle *h, ProjParams p, cudaStream_t stream) {
    if (p.M <= 0) return GVA_OK;
    if (p.K <= 0 || p.K % (16 * kProjSlices) != 0 || p.N % 8 != 0) return GVA_ERR_UNSUPPORTED;
    int m_tiles = (std::min(p.M, kProjRows) + 15) / 16, mt = 1;
    while (mt < m_tiles) mt *= 2;
    const size_t smem = (size_t)kProjChunk * kProjRowBytes + (size_t)16 * mt * kProjALd * sizeof(float);
    if (smem > (size_t)h->smem_optin) return GVA_ERR_UNSUPPORTED;
    const bool f32 = MODE == 1 && h->cfg.cache_dtype == GVA_F32;
    const bool e4m3 = MODE == 1 && h->cfg.cache_dtype == GVA_E4M3;
    void (*fn)(ProjParams, RopeTable) = nullptr;
#define GVA_PROJ(MT_) (f32 ? project_kernel<MODE, float, MT_> : e4m3 ? project_kernel<MODE, uint8_t, MT_> : project_kernel<MODE, __nv_bfloat16, MT_>)
    switch (mt) {
        case 1: fn = GVA_PROJ(1); break;
        case 2: fn = GVA_PROJ(2); break;
        case 4: fn = GVA_PROJ(4); break;
        default: fn = GVA_PROJ(8); break;
    }
#undef GVA_PROJ
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GVA_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.N + kProjStrip - 1) / kProjStrip, kProjSlices, (p.M + kProjRows - 1) / kProjRows);
    cfg.blockDim = dim3(32 * kProjWarps);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = kProjSlices;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, fn, p, h->rope) != cudaSuccess) {
        (void)cudaGetLastError();
        return GVA_ERR_CUDA;
    }
    return GVA_OK;
}
}  // namespace

extern "C" {

int gva_input_width(const gva_handle *h) { return h ? input_width(h->cfg) : 0; }

int gva_pack_input_weights(const gva_handle *h, const float *W_q_nope, const float *W_q_rope, const float *W_v,
                           const float *W_r, const float *M, int d_model, uint16_t *W_in) {
    if (!h || !W_q_nope || !W_v || !M || !W_in || d_model <= 0) return GVA_ERR_INVALID_ARG;
    if (h->cfg.d_r > 0 && (!W_q_rope || !W_r)) return GVA_ERR_INVALID_ARG;     // (a value-only cache has no positional columns)
    const gva_config &c = h->cfg;
    const int dq = c.d_v + c.d_r, nq = c.H * dq, nv = c.G * c.d_v, N = input_width(c);
    for (int m = 0; m < d_model; ++m) {
        uint16_t *row = W_in + (size_t)m * N;
        for (int hh = 0; hh < c.H; ++hh) {
            const float *wq = W_q_nope + ((size_t)m * c.H + hh) * c.d_c;
            for (int i = 0; i < c.d_v; ++i) {            // folded content columns: (W_Q^nope M_h^T)[m][i]
                const float *mi = M + ((size_t)hh * c.d_v + i) * c.d_c;
                double acc = 0.0;
                for (int j = 0; j < c.d_c; ++j) acc += (double)wq[j] * (double)mi[j];
                row[hh * dq + i] = host_bf16_from_double(acc);
            }
            for (int r = 0; r < c.d_r; ++r)
                row[hh * dq + c.d_v + r] = host_bf16_from_double((double)W_q_rope[((size_t)m * c.H + hh) * c.d_r + r]);
        }
        for (int i = 0; i < nv; ++i) row[nq + i] = host_bf16_from_double((double)W_v[(size_t)m * nv + i]);
        for (int r = 0; r < c.d_r; ++r) row[nq + nv + r] = host_bf16_from_double((double)W_r[(size_t)m * c.d_r + r]);
    }
    return GVA_OK;
}

int gva_pack_bf16(const float *src, uint16_t *dst, size_t n) {
    if (!src || !dst) return GVA_ERR_INVALID_ARG;
    for (size_t i = 0; i < n; ++i) dst[i] = host_bf16_from_double((double)src[i]);
    return GVA_OK;
}

int gva_project_in(gva_handle *h, const gva_cache *cache, const float *x, const void *W_in, int d_model,
                   const int32_t *pos, float *q_abs, int B, int32_t *dev_status, void *stream) {
    if (!h || !cache || B < 0 || d_model <= 0) return GVA_ERR_INVALID_ARG;
    if (B == 0) return GVA_OK;
    if (!x || !W_in || !pos || !q_abs || !cache->v_pool || (h->cfg.d_r > 0 && !cache->kr_pool)) return GVA_ERR_INVALID_ARG;
    if (cache->num_pages <= 0 || cache->max_pages_per_seq <= 0) return GVA_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(W_in, 16) || !aligned(q_abs, 8) || !aligned(cache->v_pool, 16) ||
        !aligned(cache->kr_pool, 16))
        return GVA_ERR_INVALID_ARG;
    const gva_config &c = h->cfg;
    ProjParams p;
    std::memset(&p, 0, sizeof(p));
    p.A = x; p.W = static_cast<const uint16_t *>(W_in);
    p.M = B; p.K = d_model; p.N = input_width(c);
    p.q_abs = q_abs; p.v_pool = cache->v_pool; p.kr_pool = cache->kr_pool;
    p.block_table = cache->block_table; p.pos = pos; p.dev_status = dev_status;
    p.H = c.H; p.G = c.G; p.d_v = c.d_v; p.d_r = c.d_r; p.P = c.page_size;
    p.num_pages = cache->num_pages; p.max_pages = cache->max_pages_per_seq;
    return launch_project<1>(h, p, static_cast<cudaStream_t>(stream));
}

int gva_project_out(gva_handle *h, const float *attn, const void *W_o, int d_model, float *y, int B, void *stream) {
    if (!h || B < 0 || d_model <= 0) return GVA_ERR_INVALID_ARG;
    if (B == 0) return GVA_OK;
    if (!attn || !W_o || !y) return GVA_ERR_INVALID_ARG;
    if (!aligned(attn, 16) || !aligned(W_o, 16) || !aligned(y, 8)) return GVA_ERR_INVALID_ARG;
    ProjParams p;
    std::memset(&p, 0, sizeof(p));
    p.A = attn; p.W = static_cast<const uint16_t *>(W_o);
    p.M = B; p.K = h->cfg.H * h->cfg.d_v; p.N = d_model;
    p.Y = y;
    return launch_project<0>(h, p, static_cast<cudaStream_t>(stream));
}

int gva_layer_step(gva_handle *h, const gva_cache *cache, const float *x, const void *W_in, const void *W_o, int d_model,
                   const int32_t *pos, const int32_t *seq_lens, float *q_abs, float *attn, float *y, void *workspace,
                   size_t workspace_bytes, int B, int max_seq_len, int num_splits, int32_t *dev_status, void *stream) {
    // the decode launch's host-side checks first: an error return then means the cache was not advanced
    int rc = decode_impl(h, cache, q_abs, seq_lens, attn, nullptr, workspace, workspace_bytes, B, max_seq_len, num_splits,
                         dev_status, stream, 0, nullptr, 1, true);
    if (rc != GVA_OK) return rc;
    rc = gva_project_in(h, cache, x, W_in, d_model, pos, q_abs, B, dev_status, stream);
    if (rc != GVA_OK) return rc;
    // (the decode kernel starts early behind the input projection, as it does behind the front kernel of gva_decode_step)
    rc = decode_impl(h, cache, q_abs, seq_lens, attn, nullptr, workspace, workspace_bytes, B, max_seq_len, num_splits,
                     dev_status, stream, 1, pos);
    if (rc != GVA_OK) return rc;
    return gva_project_out(h, attn, W_o, d_model, y, B, stream);
}

int gva_last_num_splits(const gva_handle *h) { return h ? h->last_num_splits : 0; }
int gva_last_kernel(const gva_handle *h) { return h ? h->last_kernel : 0; }
int gva_last_tile_tokens(const gva_handle *h) { return h ? h->last_tile : 0; }

#ifdef GVA_TRACE
// Development builds only: copies the in-kernel timeline stamps (kTrCalls x kTrSlots) to the host and clears them
// (synchronises the device).
int gva_debug_trace(unsigned long long *out) {
    unsigned long long init[kTrCalls * kTrSlots];
    if (cudaDeviceSynchronize() != cudaSuccess) return GVA_ERR_CUDA;
    if (cudaMemcpyFromSymbol(out, g_trace, sizeof(init)) != cudaSuccess) return GVA_ERR_CUDA;
    for (int i = 0; i < kTrCalls * kTrSlots; ++i) init[i] = (i & 1) ? 0ull : ~0ull;
    if (cudaMemcpyToSymbol(g_trace, init, sizeof(init)) != cudaSuccess) return GVA_ERR_CUDA;
    return GVA_OK;
}
#endif

const char *gva_status_string(int status) {
    switch (status) {
        case GVA_OK: return "ok";
        case GVA_ERR_INVALID_ARG: return "invalid argument";
        case GVA_ERR_UNSUPPORTED: return "unsupported shape, dtype or page size";
        case GVA_ERR_WORKSPACE: return "workspace missing or too small";
        case GVA_ERR_CUDA: return "CUDA call failed";
        case GVA_ERR_BAD_PAGE: return "block-table entry outside the page pool";
        case GVA_ERR_SEQ_LEN: return "sequence length or position outside the block table";
        case GVA_ERR_TIMEOUT: return "bounded wait on an asynchronous copy expired";
        case GVA_ERR_STATIC_LIMIT: return "request exceeds the built-in scratch of gva_decode_static";
        default: return "unknown status";
    }
}

}  // extern "C"
