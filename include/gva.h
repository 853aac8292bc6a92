/*
 * gva.h -- C ABI of the B200 (sm_100a) Grouped Value Attention decode library.
 *
 * One decode step of GVA with decoupled RoPE (Algorithm 1 of the paper) is three calls:
 *
 *   gva_absorb_query   q~_h = q^nope_h M_h^T  and  q^rope_h <- q^rope_h R_t^T      (Eq. absorb; Alg. 1)
 *   gva_append_cache   V_{1:t,g} <- [V_{1:t-1,g}; v_{t,g}],  k^rope_t = (.) R_t^T  (Eq. krope;  Alg. 1)
 *   gva_decode         s_j = q~_h v_{j,g(h)}^T + q^rope_h (k^rope_j)^T,
 *                      o_h = softmax(s / sqrt(d_qk)) V_{1:t,g(h)},  d_qk = d_c + d_r   (Section 3.3; Alg. 1)
 *
 * plus gqa_decode, a matched GQA decode over cached K and V (Section 2 / Section 3.4), built the
 * same way, as the reference point for the cache-bytes comparison N_GVA/N_GQA = 1/2 + d_r/(2 G d_h).
 *
 * Names: d_v = value width (paper d_h), d_c = content-key width (paper d_n), d_r = RoPE width,
 * H query heads, G value groups, head h reads group g(h) = h / (H/G).
 *
 * Conventions
 *   - All pointers are DEVICE pointers unless a parameter is marked [host].  The library allocates
 *     no device memory, keeps no caller pointer after a call returns, and never synchronises: every
 *     call enqueues work on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - Weights (the maps M, the packed projections W_in and W_o) are constants to the kernels: gva_absorb_query,
 *     gva_decode_step and the projections are launched as programmatic dependents of the kernel that precedes them in
 *     the stream and request their weights before they wait for that kernel's completion (all other inputs are read
 *     after the wait).  The kernel enqueued immediately before such a call must therefore not be the one that writes
 *     the weights it uses: write them by a copy, or by any earlier kernel.  (The library's own kernels never write weights.)
 *   - Return value: a gva_status detected on the host before/at launch.  Conditions only the device
 *     can see (a page id outside [0, num_pages), a sequence longer than its block table) are
 *     recorded once in *dev_status (caller-zeroed int32 on the device; may be NULL) as
 *     code | (sequence_index << 8); the offending work is skipped and the kernel ends normally.
 *   - RoPE: pairs (2i, 2i+1) of the d_r-wide slice are rotated by the angle pos * base^(-2i/d_r)
 *     (y[2i] = x[2i] cos a - x[2i+1] sin a, y[2i+1] = x[2i] sin a + x[2i+1] cos a), evaluated in fp64.
 *   - Cache layout ("pools"): v_pool [num_pages][G][page_size][d_v], kr_pool [num_pages][page_size][d_r],
 *     element type = cfg.cache_dtype.  Logical page j of sequence b is block_table[b*max_pages_per_seq + j];
 *     block_table == NULL means contiguous: page j of sequence b is b*max_pages_per_seq + j.
 *     Slots at or beyond seq_lens[b] and block-table entries beyond ceil(seq_lens[b]/page_size) are never
 *     read by gva_decode (they may hold NaN / -1).
 */
#ifndef GVA_H_
#define GVA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GVA_OK = 0,
    GVA_ERR_INVALID_ARG = 1,  /* null pointer, negative size, misaligned pointer                         */
    GVA_ERR_UNSUPPORTED = 2,  /* shape / dtype / page size outside the instantiated kernels              */
    GVA_ERR_WORKSPACE = 3,    /* workspace smaller than gva_decode_workspace_bytes()                     */
    GVA_ERR_CUDA = 4,         /* a CUDA runtime/driver call failed (launch error, no sm_100 device, ...) */
    GVA_ERR_BAD_PAGE = 5,     /* [device] block-table entry outside [0, num_pages) in the live range     */
    GVA_ERR_SEQ_LEN = 6,      /* [device] seq_len < 0 or beyond max_pages_per_seq * page_size            */
    GVA_ERR_TIMEOUT = 7,      /* [device] a bounded wait on an asynchronous copy expired                 */
    GVA_ERR_STATIC_LIMIT = 8  /* gva_decode_static: the request needs more than GVA_STATIC_SCRATCH_BYTES  */
} gva_status;

/* Element type of the cache pools.  GVA_E4M3 stores every cache element as one byte (sign, 4 exponent bits with bias 7,
 * 3 mantissa bits; no infinities, 0x7F / 0xFF = NaN, largest finite 448): appends round to nearest even and saturate
 * at +-448, decode widens the codes exactly and computes as for the other types.  The paper stores 16-bit caches; the
 * 8-bit cache is this library's extension of its byte accounting (Section 3.4) and halves the bytes per token again.
 * It is built for (d_v, d_r) = (64, 16), (64, 0), (128, 32), (128, 0), G <= 8, pages of a multiple of 64 tokens, with the
 * tensor-core kernel only:
 * gva_absorb_query, gva_append_cache, gva_append_chunk, gva_decode, gva_decode_step, gva_decode_step_host,
 * gva_decode_static, gqa_decode (keys and values as e4m3 codes), the projections, gva_layer_step and (with a positional
 * slice, d_r > 0) gva_decode_tokens / gva_decode_tokens_ragged serve it, and so do gva_prefill and gva_decode_multi (the
 * byte tiles are widened to f16 in shared memory; queries and weights are then f16 instead of bf16). */
typedef enum { GVA_F32 = 0, GVA_BF16 = 1, GVA_E4M3 = 2 } gva_dtype;

/* Which decode kernel gva_decode launches.  AUTO = tensor-core kernel when the cache is bf16 or e4m3,
 * CUDA-core (FMA) kernel for an f32 cache.  FMA / MMA force one (MMA with an f32 cache and
 * FMA with an e4m3 cache are GVA_ERR_UNSUPPORTED). */
typedef enum { GVA_KERNEL_AUTO = 0, GVA_KERNEL_FMA = 1, GVA_KERNEL_MMA = 2 } gva_kernel;

typedef struct {
    int32_t H, G;          /* query heads, value groups; H % G == 0 and H/G == 4                          */
    int32_t d_v;           /* value width: 64 or 128                                                      */
    int32_t d_c;           /* content-key width (only gva_absorb_query uses it): 1..256                   */
    int32_t d_r;           /* RoPE width: 16 or 24 with d_v = 64 (the paper's two tested widths), 32 with d_v = 128;
                              0 = value-only cache without a positional slice (Section 3.4: a cache of values alone is
                              half of matched GQA's): kr_pool, q_r and kr_new are then unused and may be NULL, scale = 1/sqrt(d_c) */
    int32_t page_size;     /* tokens per page, a multiple of 32                                           */
    int32_t cache_dtype;   /* gva_dtype                                                                   */
    int32_t kernel;        /* gva_kernel                                                                  */
    double rope_base;      /* 10000.0                                                                     */
    float softmax_scale;   /* 0 => 1/sqrt(d_c + d_r)                                                      */
    int32_t reserved;      /* set to 0                                                                    */
} gva_config;

typedef struct {
    void *v_pool;               /* [num_pages][G][page_size][d_v]   16-byte aligned                        */
    void *kr_pool;              /* [num_pages][page_size][d_r]      16-byte aligned                        */
    const int32_t *block_table; /* [B][max_pages_per_seq] or NULL (contiguous)                             */
    int32_t num_pages;
    int32_t max_pages_per_seq;
} gva_cache;

typedef struct {
    void *k_pool;               /* [num_pages][G][page_size][d_h]  keys, already rotated                    */
    void *v_pool;               /* [num_pages][G][page_size][d_h]                                           */
    const int32_t *block_table;
    int32_t num_pages;
    int32_t max_pages_per_seq;
} gqa_cache;

typedef struct gva_handle gva_handle; /* opaque host-side state: config, device properties, last launch geometry */

/* Create / destroy a handle for one head configuration on one device.  Validates cfg
 * (GVA_ERR_UNSUPPORTED / GVA_ERR_INVALID_ARG), checks that `device` is compute capability 10.x
 * (GVA_ERR_CUDA otherwise) and raises the kernels' shared-memory limits.  Makes `device` current.
 *
 * One handle, one stream at a time.  Besides its host-side state a handle owns a few words of DEVICE-side
 * scheduling state inside the library image (the counters through which the thread blocks of a decode
 * kernel share out the tail of the cache stream).  Decode calls on one handle -- gva_decode, gqa_decode,
 * gva_decode_step(_host), gva_decode_static, gva_decode_tokens, gva_layer_step -- must therefore be
 * stream-ordered with respect to one another: issue them on one stream, or order the streams with events.
 * Two such calls that may overlap on the GPU race on those words even if their workspaces differ (wrong
 * partition of the work, hence wrong results; never a fault).  Use one handle per concurrent stream; handles
 * are cheap (no device allocation).  The handle is not thread-safe either: one host thread at a time.
 * gva_destroy only after the last call on the handle has finished on the device. */
int gva_create(gva_handle **out, const gva_config *cfg, int device);
int gva_destroy(gva_handle *h);

/* Bytes of scratch gva_decode / gqa_decode need for B sequences of at most max_seq_len tokens with
 * the given num_splits (same meaning as in gva_decode).  Holds the split-KV partial results
 * (unnormalised output, running max and sum per partition and head).  0 on invalid arguments. */
size_t gva_decode_workspace_bytes(const gva_handle *h, int B, int max_seq_len, int num_splits);

/* Eq. absorb and the query-side rotation of Algorithm 1.
 *   q_c   [B][H][d_c] f32   content ("nope") query slices
 *   q_r   [B][H][d_r] f32   positional query slices, unrotated
 *   M     [H][d_v][d_c] f32 reconstruction maps, row-major (M_h in R^{d_h x d_n}; K_h = V_g(h) M_h)
 *   q_pos [B] i32           query positions t (0-based)
 *   q_abs [B][H][d_v+d_r] f32 out:  [:d_v] = q_c M_h^T  (q~[i] = sum_j q_c[j] M_h[i][j]),
 *                                   [d_v:] = q_r R_t^T */
int gva_absorb_query(gva_handle *h, const float *q_c, const float *q_r, const float *M,
                     const int32_t *q_pos, float *q_abs, int B, void *stream);

/* Algorithm 1's cache append for one new token per sequence.
 *   v_new  [B][G][d_v] f32   new value rows;  kr_new [B][d_r] f32 unrotated positional key (x_t W_r)
 *   pos    [B] i32           0-based position t of the new token
 * Writes, for each b, rows (page = block_table[b][t/page_size], slot = t % page_size):
 *   v_pool[page][g][slot][:] = cast(v_new[b][g][:]),  kr_pool[page][slot][:] = cast(kr_new[b] R_t^T)
 * cast = round-to-nearest-even to the cache dtype (from the fp64 rotation for k^rope); no other byte
 * of the pools changes.  pos < 0 or beyond the block table -> GVA_ERR_SEQ_LEN in *dev_status, bad
 * page id -> GVA_ERR_BAD_PAGE; that sequence is skipped. */
int gva_append_cache(gva_handle *h, const gva_cache *cache, const float *v_new, const float *kr_new,
                     const int32_t *pos, int B, int32_t *dev_status, void *stream);

/* Decode attention over the cache (the score and softmax-value lines of Algorithm 1) for B
 * sequences, query heads sharing each value group's stream.
 *   q_abs    [B][H][d_v+d_r] f32  from gva_absorb_query
 *   seq_lens [B] i32              number of cached tokens attended (positions 0..seq_len-1)
 *   out      [B][H][d_v] f32      o_h;  seq_len == 0 gives 0
 *   lse      [B][H] f32 or NULL   natural log of sum_j exp(scale * s_j); -inf for seq_len == 0
 *   workspace / workspace_bytes   scratch of at least gva_decode_workspace_bytes(h, B, max_seq_len, num_splits),
 *                                 256-byte aligned; contents are overwritten; calls sharing it must be
 *                                 stream-ordered
 *   max_seq_len                   upper bound on seq_lens[] (sizes the launch; a longer sequence is
 *                                 still computed correctly as long as it fits its block table)
 *   num_splits                    0: the cache stream is cut into equal contiguous ranges of tiles, one
 *                                 per resident thread block (ranges may cross sequence boundaries);
 *                                 n >= 1: every sequence is cut into exactly n ranges.
 * Partial results are merged by log-sum-exp weights in a second kernel.  For fixed arguments the
 * result is bitwise reproducible from run to run.  Calls on one handle must be stream-ordered (see gva_create).
 * The call may be captured into a CUDA graph (after one call outside the capture, which sizes the handle's scheduling
 * state) and replayed with different contents of its device buffers: every call leaves the scheduling words as it
 * found them, and nothing on the device depends on the call's number changing between replays. */
int gva_decode(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens,
               float *out, float *lse, void *workspace, size_t workspace_bytes, int B, int max_seq_len,
               int num_splits, int32_t *dev_status, void *stream);

/* gva_decode for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * entry point exists for the library's users, not for the method.)
 *
 * Who this is for: code that runs where cudaMalloc is off limits -- inside a serving loop whose memory
 * pool was sized and frozen at start-up, under a framework allocator that forbids side allocations, or
 * in a plug-in that is handed tensors but no allocator.  Such callers cannot provide the split-KV
 * workspace gva_decode asks for, so here the partial results live in a fixed array compiled into the
 * library (GVA_STATIC_SCRATCH_BYTES of device memory, held by every GPU that loads the library until
 * the process exits).  Inputs and outputs are still the caller's, with the same meaning, layout and
 * error rules as gva_decode; neither this call nor anything it uses calls cudaMalloc, cudaFree or an
 * allocating library routine.
 *
 *  - Limit: if gva_decode_workspace_bytes(h, B, max_seq_len, num_splits) exceeds
 *    GVA_STATIC_SCRATCH_BYTES the call launches nothing and returns GVA_ERR_STATIC_LIMIT.  At num_splits = 0
 *    the need grows with the batch (one partial record per sequence on top of a few per thread block), not
 *    with the context length: on a B200 the five workloads of the benchmark take 2.5 to 5.5 MB (for example
 *    B = 32 sequences of 32768 tokens, H = 16, d_v = 64: 5.1 MB; B = 64, H = 32, d_v = 128: 3.5 MB), and
 *    H = 16, d_v = 64 fits up to about B = 2700.  With num_splits = n the need is B * n records of
 *    H * (d_v + 2) * 4 bytes each.
 *  - Set-up: the first call on each device looks up the array's device address (once per device; the
 *    handle's device must be the current device, otherwise GVA_ERR_INVALID_ARG).  Make that first
 *    call outside any stream capture.
 *  - Sharing: every call on a device uses the same array, and it keeps whatever the previous call left.
 *    Nothing needs clearing -- each call writes every word it later reads -- but two calls that may run
 *    at the same time on one GPU (different streams, different handles, different threads) race on it:
 *    keep calls to this entry point stream-ordered per device. */
#define GVA_STATIC_SCRATCH_BYTES (16u << 20)
int gva_decode_static(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens,
                      float *out, float *lse, int B, int max_seq_len, int num_splits, int32_t *dev_status,
                      void *stream);

/* Matched GQA decode (two cached streams): s_j = q_h K_{j,g(h)}^T / sqrt(d_h), o_h = softmax(s) V_{g(h)},
 * with d_h = cfg.d_v, q [B][H][d_h] f32 already rotated, K cached already rotated.  Same paging,
 * splitting, workspace and error rules as gva_decode.  cfg.d_c, cfg.d_r and cfg.softmax_scale are
 * ignored (scale = 1/sqrt(d_h)). */
int gqa_decode(gva_handle *h, const gqa_cache *cache, const float *q, const int32_t *seq_lens, float *out,
               float *lse, void *workspace, size_t workspace_bytes, int B, int max_seq_len, int num_splits,
               int32_t *dev_status, void *stream);

/* One whole decode step on device buffers: the same results, bit for bit, as gva_absorb_query ->
 * gva_append_cache -> gva_decode called in that order (Algorithm 1 from the split queries to the
 * per-head outputs), in two launches instead of four: absorb and append run in one kernel, and the
 * decode kernel starts its bookkeeping and its first cache loads while that kernel computes.
 *   pos      [B] i32  position t of the new token: the append slot and the query position
 *   seq_lens [B] i32  tokens attended (normally t + 1, so the query sees its own token)
 *   q_abs    [B][H][d_v+d_r] f32  written by the call (the absorbed queries), then read by the decode
 *   other arguments as in the three separate calls.
 * Because the decode kernel reads seq_lens, pos, the block table and cache tiles other than the one
 * receiving the new token before the fused front kernel has finished, those must not be outputs of
 * that same call; everything enqueued on the stream before the call is complete before any of it is read. */
int gva_decode_step(gva_handle *h, const gva_cache *cache, const float *M, const float *q_c, const float *q_r,
                    const float *v_new, const float *kr_new, const int32_t *pos, const int32_t *seq_lens,
                    float *q_abs, float *out, float *lse, void *workspace, size_t workspace_bytes, int B,
                    int max_seq_len, int num_splits, int32_t *dev_status, void *stream);

/* One whole decode step (Algorithm 1 from the split queries to the per-head outputs) for callers whose
 * per-step tensors live in HOST memory: copies the step's inputs to the device, runs
 * gva_decode_step, and copies the outputs back, all enqueued on
 * `stream`; the caller synchronises the stream before reading out_host.  The cache and the maps M stay
 * resident on the device (they are state, not per-step input).
 *   [host] q_c_host [B][H][d_c], q_r_host [B][H][d_r], v_new_host [B][G][d_v], kr_new_host [B][d_r] f32,
 *          pos_host [B] i32 (position t of the new token = query position), seq_lens_host [B] i32
 *          (tokens attended, normally t + 1).  If the four float inputs and out_host are all pinned
 *          (page-locked, device-mapped) memory the kernels read and write them in place over the
 *          interconnect and only pos and seq_lens are brought to the device (by a one-block kernel when they are
 *          pinned too, else by two copies); otherwise every buffer is staged through
 *          `scratch` with cudaMemcpyAsync (pageable memory makes those copies synchronous).
 *   [host] out_host [B][H][d_v] f32
 *   M                device, as in gva_absorb_query
 *   scratch          device, at least gva_step_scratch_bytes(h, B, max_seq_len, num_splits) bytes, 256-byte aligned;
 *                    holds the staged inputs, q_abs, out and the decode workspace.
 * Bytes moved per call: host->device B*(H*(d_c+d_r) + G*d_v + d_r)*4 + 8*B, device->host B*H*d_v*4. */
size_t gva_step_scratch_bytes(const gva_handle *h, int B, int max_seq_len, int num_splits);
int gva_decode_step_host(gva_handle *h, const gva_cache *cache, const float *M, const float *q_c_host,
                         const float *q_r_host, const float *v_new_host, const float *kr_new_host,
                         const int32_t *pos_host, const int32_t *seq_lens_host, float *out_host, void *scratch,
                         size_t scratch_bytes, int B, int max_seq_len, int num_splits, int32_t *dev_status,
                         void *stream);

/* ---- The projections around the attention (Algorithm 1: q_t = x_t W_Q, v_t = x_t W_V, k^rope_t = (x_t W_r) R_t^T;
 * then the heads side by side through the output projection), with the maps folded into the query projection:
 * because M_h is fixed at inference, q~_h = (x W_Q^{nope,h}) M_h^T = x (W_Q^{nope,h} M_h^T)  (Eq. absorb), so
 * one product with a packed weight matrix yields the absorbed queries directly and gva_absorb_query drops out.
 *
 * Packed input projection W_in: bf16 [d_model][N_in], N_in = gva_input_width() = H*(d_v+d_r) + G*d_v + d_r,
 * columns per head h: d_v folded content columns (W_Q^{nope,h} M_h^T), then d_r positional-query columns;
 * then the G*d_v value columns; then the d_r positional-key columns.  d_model must be a multiple of 128. */
int gva_input_width(const gva_handle *h);

/* [host] Offline packing of one layer's input projection: folds the maps in fp64 and rounds every entry once to
 * bf16.  W_q_nope [d_model][H][d_c], W_q_rope [d_model][H][d_r], W_v [d_model][G][d_v], W_r [d_model][d_r],
 * M [H][d_v][d_c] f32 (host); W_in [d_model][N_in] bf16 bit patterns (host, caller uploads it).  With a value-only
 * cache (d_r = 0) there are no positional columns: W_q_rope and W_r are unused and may be NULL. */
int gva_pack_input_weights(const gva_handle *h, const float *W_q_nope, const float *W_q_rope, const float *W_v,
                           const float *W_r, const float *M, int d_model, uint16_t *W_in);
/* [host] f32 -> bf16 bit patterns, nearest even (for the output projection W_o). */
int gva_pack_bf16(const float *src, uint16_t *dst, size_t n);

/* x [B][d_model] f32 -> q_abs [B][H][d_v+d_r] f32 (positional slice rotated at pos[b]) and the cache append of the
 * new token at pos[b], in one kernel.  The appended rows are bit for bit what gva_append_cache writes when it is given
 * the kernel's own f32 products as v_new / kr_new (value rows rounded once to the cache dtype, k^rope rotated in fp64
 * and rounded once); against products accumulated in higher precision they can differ by one unit in the last place
 * of the cache dtype.  Same device-side error rules as gva_append_cache. */
int gva_project_in(gva_handle *h, const gva_cache *cache, const float *x, const void *W_in, int d_model,
                   const int32_t *pos, float *q_abs, int B, int32_t *dev_status, void *stream);
/* attn [B][H*d_v] f32 (heads concatenated, as gva_decode writes them) x W_o bf16 [H*d_v][d_model] -> y [B][d_model] f32. */
int gva_project_out(gva_handle *h, const float *attn, const void *W_o, int d_model, float *y, int B, void *stream);
/* A whole layer's decode step from the hidden state: gva_project_in -> gva_decode -> gva_project_out. */
int gva_layer_step(gva_handle *h, const gva_cache *cache, const float *x, const void *W_in, const void *W_o,
                   int d_model, const int32_t *pos, const int32_t *seq_lens, float *q_abs, float *attn, float *y,
                   void *workspace, size_t workspace_bytes, int B, int max_seq_len, int num_splits,
                   int32_t *dev_status, void *stream);

/* ---- Several new tokens per sequence: prefill and chunked prefill (the paper's multi-token form: ordinary causal
 * attention whose scores keep the content + positional split, Section 3.3 and the remark after Algorithm 1), computed in the
 * absorbed form of Eq. absorb.  Sequence b has ctx_lens[b] tokens cached already and q_len_b = cu_q[b+1] - cu_q[b]
 * new tokens; new token i of sequence b is input row cu_q[b] + i, sits at position t = ctx_lens[b] + i and attends
 * to positions 0..t.  The order of calls is Algorithm 1's, once per chunk instead of once per token:
 *   gva_absorb_query(B := n_q, q_pos[row] = position of the row)  ->  gva_append_chunk  ->  gva_prefill.
 *   cu_q [B+1] i32 (cu_q[0] = 0, non-decreasing), ctx_lens [B] i32, n_q = cu_q[B] rows in all. */

/* Algorithm 1's append for every new token of the chunk: row n of v_new [n_q][G][d_v] / kr_new [n_q][d_r] (unrotated)
 * is written at its position exactly as gva_append_cache writes one token (same rounding, same error rules). */
int gva_append_chunk(gva_handle *h, const gva_cache *cache, const float *v_new, const float *kr_new,
                     const int32_t *cu_q, const int32_t *ctx_lens, int B, int n_q, int32_t *dev_status, void *stream);

/* Causal attention of the chunk over the cache, which must already hold the chunk's own tokens.
 *   q_abs [n_q][H][d_v+d_r] f32  from gva_absorb_query;  out [n_q][H][d_v] f32;  lse [n_q][H] f32 or NULL
 *   max_q_len                    upper bound on the q_len_b (sizes the launch; longer chunks are cut off)
 * bf16 or e4m3 cache, page_size a multiple of 64, (d_v, d_r) = (64, 16), (64, 24) (bf16 only), (128, 32), (64, 0) or
 * (128, 0); otherwise GVA_ERR_UNSUPPORTED.
 * Runs on the tensor cores with bf16 operands (the absorbed query and the softmax weights are rounded to bf16,
 * accumulation is f32), so results carry bf16-level error: |out - exact| <= 2e-2 for unit-variance data.
 * Device-side errors as in gva_decode; a thread block that meets one stops and leaves its rows of out unwritten. */
int gva_prefill(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q,
                const int32_t *ctx_lens, float *out, float *lse, int B, int max_q_len, int32_t *dev_status,
                void *stream);

/* Decode of several new tokens per sequence over a long cached context (speculative / multi-token decode; not in the
 * paper -- Algorithm 1 applied to q_len_b tokens at once, i.e. gva_prefill's computation) with split-KV: every block of
 * 32 query tokens is handled by several thread blocks, each over a contiguous range of 64-token tiles, and a second
 * kernel merges their partial results by log-sum-exp weights, so that small batches still fill the GPU.
 *   arguments as gva_prefill, plus
 *   n_q                          cu_q[B]: query rows in all (sizes the merge)
 *   max_seq_len                  upper bound on ctx_lens[b] + q_len_b
 *   num_splits                   0 = enough splits for two thread blocks per SM; n >= 1 = exactly n (at most one per tile, 64)
 *   workspace / workspace_bytes  at least gva_decode_multi_workspace_bytes(...) bytes, 256-byte aligned
 * Same support, tolerance and error rules as gva_prefill. */
size_t gva_decode_multi_workspace_bytes(const gva_handle *h, int B, int n_q, int max_q_len, int max_seq_len,
                                        int num_splits);
int gva_decode_multi(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q,
                     const int32_t *ctx_lens, float *out, float *lse, void *workspace, size_t workspace_bytes, int B,
                     int n_q, int max_q_len, int max_seq_len, int num_splits, int32_t *dev_status, void *stream);

/* Decode of q_len = 2 .. 8 new tokens per sequence at the single-token kernel's cache-stream rate (speculative /
 * multi-token decode; not in the paper -- Algorithm 1 applied to q_len tokens at once).  The split-KV tensor-core decode
 * kernel of gva_decode carries the 4 * q_len (head, token) pairs of a value group as its MMA columns, so the cache is
 * streamed once for all of them.  Every sequence has exactly q_len new tokens, already appended.
 *   q_abs    [B * q_len][H][d_v+d_r] f32  row b * q_len + i = new token i of sequence b (from gva_absorb_query)
 *   seq_lens [B] i32                      tokens attended by the LAST new token; new token i attends seq_lens[b] - (q_len-1-i)
 *   out      [B * q_len][H][d_v] f32, lse [B * q_len][H] f32 or NULL
 *   workspace                             at least gva_decode_tokens_workspace_bytes(...) bytes, 256-byte aligned
 * q_len 2 .. 4: bf16 cache with (d_v, d_r) = (64, 16), (64, 24) (pages of a multiple of 64 tokens), (64, 0), (128, 32) or
 * (128, 0), and the e4m3 cache with a positional slice; q_len 5 .. 8: bf16 cache with d_v = 64, d_r = 16, 24 or 0, G <= 4
 * and pages of a multiple of 64 tokens; tensor-core kernel only; otherwise GVA_ERR_UNSUPPORTED.  The queries enter the score product as two bf16 numbers each (hi + lo), the
 * softmax weights as one (the 8-bit cache: f16 instead of bf16), accumulation is f32: |out - exact| <= 2e-2 whatever
 * the size of the scores. */
size_t gva_decode_tokens_workspace_bytes(const gva_handle *h, int B, int q_len, int max_seq_len, int num_splits);
int gva_decode_tokens(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *seq_lens, float *out,
                      float *lse, void *workspace, size_t workspace_bytes, int B, int q_len, int max_seq_len,
                      int num_splits, int32_t *dev_status, void *stream);

/* The same with a different number of new tokens per sequence (a batch in which some sequences verify eight draft
 * tokens, some two, some none): sequence b has q_len_b = cu_q[b+1] - cu_q[b] new tokens, 0 <= q_len_b <= max_q_len <= 8,
 * already appended; its rows of q_abs / out / lse are cu_q[b] .. cu_q[b+1] - 1 (cu_q [B + 1] i32, cu_q[0] = 0,
 * non-decreasing).  seq_lens[b] = tokens attended by the last new token of b; new token i attends
 * seq_lens[b] - (q_len_b - 1 - i).  Workspace: gva_decode_tokens_workspace_bytes(h, B, max(max_q_len, 2), ...).
 * Caches and shapes as gva_decode_tokens for the given max_q_len.  Same accuracy. */
int gva_decode_tokens_ragged(gva_handle *h, const gva_cache *cache, const float *q_abs, const int32_t *cu_q,
                             const int32_t *seq_lens, float *out, float *lse, void *workspace, size_t workspace_bytes, int B,
                             int max_q_len, int max_seq_len, int num_splits, int32_t *dev_status, void *stream);

/* Geometry of the most recent gva_decode / gqa_decode launch on this handle (reporting only):
 * number of split-KV partitions launched (thread blocks of the decode kernel). */
int gva_last_num_splits(const gva_handle *h);
/* 1 = CUDA-core (FMA) kernel, 2 = tensor-core (MMA) kernel, 0 = none yet. */
int gva_last_kernel(const gva_handle *h);
/* Tokens per tile of the kernel chosen by the last launch (the unit in which ranges are cut). */
int gva_last_tile_tokens(const gva_handle *h);

const char *gva_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GVA_H_ */
