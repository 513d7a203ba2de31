/*
 * carnator.h -- C ABI of the block-sparse attention hot path (CUDA, sm_100a).
 *
 * The library executes one self-attention layer of a video diffusion
 * transformer the way the paper's cross-request reuse does on a cache hit:
 * the target request's own Q, K and V are used, but only the (query block,
 * key block) pairs recorded in a historical request's block-connectivity mask
 * are evaluated; query blocks flagged as target-specific are evaluated
 * densely.  A companion call builds such a mask from block-pooled Q.K^T scores
 * when a request's computation is written into the cache.
 *
 * General conventions (every entry point):
 *   - Unless a parameter is documented as a HOST pointer, every data pointer is
 *     a DEVICE pointer owned by the caller.  The library never allocates or
 *     frees device memory; scratch space is passed in as a workspace whose size
 *     the *_workspace_bytes queries return.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream).  Only carnator_query_status and the *_host calls
 *     synchronise.
 *   - Arguments are validated on the host before any launch.  A failed call
 *     launches nothing and returns an error code; nothing aborts or throws.
 *   - Q, K, V, O are bf16 with the head dimension contiguous; the element
 *     strides of the (batch, head, token) axes are given in the shape record and
 *     must be multiples of 8 elements (16 bytes); base pointers 16-byte aligned.
 *     A batch or head stride of 0 shares one tensor over that axis (e.g. K and V
 *     common to all heads); such inputs run on the portable attention kernel.
 *   - Token order: text tokens first (n_text of them), then video tokens
 *     flattened frame-major (t, then grid row, then grid column).  Blocks are
 *     contiguous runs of block_q / block_k tokens of that order; the last block
 *     may be partial.  Buffers may hold more than N rows; rows >= N are never
 *     read as keys and never written.
 *   - Mask bytes and recompute bytes: non-zero = keep / recompute.
 *   - Attention is bidirectional softmax attention; LSE is the natural log of
 *     the sum of exp(scaled scores) over the keys a query sees.  A query that
 *     sees no key gets O = 0 and LSE = -inf.
 *   - There is no CPU fallback: on a machine without an sm_100 device the
 *     compute calls return CARNATOR_ERR_UNSUPPORTED.
 */
#ifndef CARNATOR_H_
#define CARNATOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum carnator_status {
    CARNATOR_OK = 0,
    CARNATOR_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, misaligned pointer or stride, n_text + T*Hg*Wg != N */
    CARNATOR_ERR_UNSUPPORTED = 2,   /* D not in {64,128}, block size not in {64,128}, too many key blocks, no sm_100 device */
    CARNATOR_ERR_WORKSPACE = 3,     /* workspace NULL, misaligned (256 B) or smaller than the matching *_workspace_bytes */
    CARNATOR_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed; see carnator_last_cuda_error */
    CARNATOR_ERR_DEVICE_TIMEOUT = 5,/* a bounded wait inside a kernel expired; the kernel drained and returned */
    CARNATOR_ERR_DEVICE_CHECK = 6   /* a device-side consistency check failed (malformed compacted lists) */
} carnator_status;

/* Which attention kernel executes the compacted lists. */
enum {
    CARNATOR_IMPL_AUTO = 0,      /* tcgen05 kernel where it supports the shape, else the portable kernel */
    CARNATOR_IMPL_PORTABLE = 1,  /* mma.sync kernel: any supported shape */
    CARNATOR_IMPL_TCGEN05 = 2    /* TMA + tcgen05/TMEM kernel: block_q = block_k = 128 and no zero K/V stride on a batch or head
                                    axis longer than 1 (a tensor shared over heads); else CARNATOR_ERR_UNSUPPORTED */
};

/* Problem description shared by all calls. */
typedef struct carnator_shape {
    int32_t B, H, N, D;             /* batch, heads, valid tokens per head, head dimension (64 or 128) */
    int32_t n_text, T, Hg, Wg;      /* n_text + T*Hg*Wg == N; latent grid T x Hg x Wg */
    int32_t block_q, block_k;       /* 64 or 128 */
    int64_t q_stride[3];            /* element strides of (batch, head, token) for Q; head dim has stride 1 */
    int64_t k_stride[3];
    int64_t v_stride[3];
    int64_t o_stride[3];
    float   softmax_scale;          /* <= 0 selects 1/sqrt(D) */
    int32_t attn_impl;              /* CARNATOR_IMPL_* */
} carnator_shape;

/* Selection rule of the connectivity builder. */
enum { CARNATOR_MODE_TOPK = 0, CARNATOR_MODE_CUMMASS = 1 };

typedef struct carnator_build_params {
    int32_t mode;                   /* CARNATOR_MODE_TOPK: keep_ratio; CARNATOR_MODE_CUMMASS: mass */
    float   keep_ratio;             /* TOPK: k = clamp(ceil(keep_ratio * n - 1e-6), 1, n) over the n candidates of a row */
    float   mass;                   /* CUMMASS: fraction of the row's pooled-softmax mass to cover, in (0, 1] */
    int32_t window_frames;          /* -1: none; r >= 0: key blocks touching frames [f_lo - r, f_hi + r] of the query block are always kept */
    int32_t text_dense;             /* 1: blocks holding a text token are dense rows and dense columns */
    int32_t count_includes_forced;  /* TOPK: 1: k counts the always-kept blocks; 0: k applies to the other candidates only */
} carnator_build_params;

/* ------------------------------------------------------------------------
 * Connectivity builder (cache-write side).
 *
 * Paper: Appendix "Reuse-Scope Implementation Details" -- self-attention is
 * partitioned into query x key blocks and, per head and query block, the
 * smallest set of key blocks covering a fixed fraction of the attention mass is
 * kept as a binary mask.  This call estimates block mass from block-pooled
 * scores: q_bar_I / k_bar_J = mean of the block's valid token rows (fp32),
 * S[I,J] = scale * <q_bar_I, k_bar_J> (fp32), then per row either the k best
 * blocks (ties: lower key-block index first) or the shortest descending prefix
 * whose softmax mass over the row reaches `mass`, in both cases together with
 * the always-kept blocks (frame window, text rows / columns).
 *
 *   Q, K   device, bf16 [B,H,>=N,D] with the strides of `shape`
 *   mask   device, uint8 [B,H,nqb,nkb] contiguous, written (1 = keep, 0 = drop)
 *   pooled_scores_opt  device, fp32 [B,H,nqb,nkb] contiguous or NULL; when given it
 *          receives S (and replaces the score area of the workspace)
 *   ws     device workspace, 256-byte aligned, >= carnator_build_workspace_bytes
 * In top-k mode with nkb <= 1024, on layers large enough to fill the GPU, the three steps run as one persistent
 * kernel (block sums and pooled scores on the tensor cores -- the means split into three bf16 terms, fp32 accumulate --
 * at HBM speed, selection on chip beside them); otherwise,
 * and in cumulative-mass mode, as three kernels with the scores held in the workspace.
 * Limits: nkb <= 4096.
 * ------------------------------------------------------------------------ */
size_t carnator_build_workspace_bytes(const carnator_shape* shape, const carnator_build_params* params);

carnator_status carnator_build_connectivity(const void* Q, const void* K,
                                            const carnator_shape* shape,
                                            const carnator_build_params* params,
                                            uint8_t* mask, float* pooled_scores_opt,
                                            void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Connectivity builder on the exact block attention mass (cache-write side).
 *
 * Paper: Appendix "Reuse-Scope Implementation Details", stated literally -- per head and query
 * block, the smallest set of key blocks covering a fixed fraction of the attention mass, where
 *   mass[I,J] = (1/|I|) * sum_{i in I} sum_{j in J} exp(s_ij - LSE_i)
 * is the share of query block I's softmax attention that falls into key block J (rows sum to 1).
 * LSE is the log-sum-exp over all keys that a dense run of carnator_sparse_attn (all-ones mask)
 * returns for the same Q and K, so this call is a second pass over Q K^T on the tensor cores
 * followed by the cumulative-mass selection (ties: lower key-block index first; the always-kept
 * blocks of `params` count towards the covered mass).
 *
 *   Q, K    device, bf16, strides of `shape`;  LSE  device, fp32 [B,H,N] contiguous, natural log
 *   params  mass, window_frames and text_dense are used; mode / keep_ratio are ignored
 *   mask    device, uint8 [B,H,nqb,nkb], written
 *   block_mass_opt  device, fp32 [B,H,nqb,nkb] or NULL; receives the masses
 *   ws      device workspace, 256-byte aligned, >= carnator_exact_workspace_bytes
 * Limits: block_q = block_k = 128, nkb <= 4096.
 * ------------------------------------------------------------------------ */
size_t carnator_exact_workspace_bytes(const carnator_shape* shape);

carnator_status carnator_build_connectivity_exact(const void* Q, const void* K, const float* LSE,
                                                  const carnator_shape* shape,
                                                  const carnator_build_params* params,
                                                  uint8_t* mask, float* block_mass_opt,
                                                  void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Sparse attention under a reused mask (cache-hit side).
 *
 * Paper: Section 3.3, "Historical Sparse-Connectivity Reuse" (the target's Q, K,
 * V are recomputed; the historical block structure decides which query-key
 * interactions are evaluated) and "Joint Reuse in Intermediate Layers" /
 * Algorithm 1 (target-specific query blocks are recomputed); latency accounting
 * of mask / index lookups: Appendix "Latency Accounting".
 *
 * Query block I of head (b,h) attends to every key of key block J iff
 * recompute_rows[b,I] != 0 or mask[b,h,I,J] != 0.
 *
 *   Q, K, V  device, bf16, strides of `shape`
 *   mask     device, uint8 [B,H,nqb,nkb] contiguous (read only)
 *   recompute_rows  device, uint8 [B,nqb] contiguous, or NULL for "none"
 *   O        device, bf16, strides o_stride; rows < N written
 *   LSE      device, fp32 [B,H,N] contiguous
 *   ws       device workspace, 256-byte aligned, >= carnator_attn_workspace_bytes
 *
 * carnator_sparse_attn = carnator_compact_mask + carnator_sparse_attn_compacted.
 * The split lets a caller compact a mask once and reuse the lists (a mask belongs
 * to one denoising step, guidance branch and layer and is the same for every
 * request that reuses that cache entry).  The workspace then carries the lists
 * between the two calls and must not be modified in between.
 *
 * carnator_compact_mask writes, per (b,h,I), the ascending list of key blocks to
 * evaluate and its length, and per (b,h) an execution order of the query blocks
 * (longest list first).
 * ------------------------------------------------------------------------ */
size_t carnator_attn_workspace_bytes(const carnator_shape* shape);

carnator_status carnator_compact_mask(const uint8_t* mask, const uint8_t* recompute_rows,
                                      const carnator_shape* shape,
                                      void* ws, size_t ws_bytes, void* stream);

carnator_status carnator_sparse_attn_compacted(const void* Q, const void* K, const void* V,
                                               const carnator_shape* shape,
                                               void* O, float* LSE,
                                               void* ws, size_t ws_bytes, void* stream);

carnator_status carnator_sparse_attn(const void* Q, const void* K, const void* V,
                                     const uint8_t* mask, const uint8_t* recompute_rows,
                                     const carnator_shape* shape,
                                     void* O, float* LSE,
                                     void* ws, size_t ws_bytes, void* stream);

/* Number of evaluated (query block, key block) pairs after compaction, summed over
 * all heads.  Synchronises `stream`.  *tiles is a HOST pointer. */
carnator_status carnator_compacted_tiles(const carnator_shape* shape, const void* ws, size_t ws_bytes,
                                         void* stream, int64_t* tiles);

/* ------------------------------------------------------------------------
 * Host-buffer forms of the two calls (end-to-end use and measurement).
 * Q/K/V/mask/recompute_rows/O/LSE/pooled scores are HOST pointers (pinned memory
 * for full copy speed) laid out contiguously: Q,K,V,O [B,H,N,D] bf16 (the strides
 * in `shape` are ignored), LSE [B,H,N], mask [B,H,nqb,nkb], recompute_rows [B,nqb].
 * `arena` is a DEVICE buffer of at least carnator_*_host_arena_bytes that holds
 * the device copies and the workspace.  The calls copy in, run, copy out and
 * synchronise `stream` before returning.
 * carnator_sparse_attn_host works through the heads in chunks of about 64 MB per
 * tensor: the copy-in of one chunk, the kernels of the previous one and the
 * copy-out of the one before run at the same time, on two copy streams that the
 * library creates once per device (first call) and keeps; the kernels run on
 * `stream`, after everything queued on it before the call.  One such call at a
 * time per process (an internal lock serialises them).  Each chunk has its own
 * workspace header inside the arena; the call returns the first failure.
 * ------------------------------------------------------------------------ */
size_t carnator_attn_host_arena_bytes(const carnator_shape* shape);

carnator_status carnator_sparse_attn_host(const void* Q, const void* K, const void* V,
                                          const uint8_t* mask, const uint8_t* recompute_rows,
                                          const carnator_shape* shape,
                                          void* O, float* LSE,
                                          void* arena, size_t arena_bytes, void* stream);

size_t carnator_build_host_arena_bytes(const carnator_shape* shape, const carnator_build_params* params);

carnator_status carnator_build_connectivity_host(const void* Q, const void* K,
                                                 const carnator_shape* shape,
                                                 const carnator_build_params* params,
                                                 uint8_t* mask,
                                                 void* arena, size_t arena_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Reuse regions, latent fusion and the region-restricted (middle-layer) attention form.
 *
 * Paper: Section 3.3 "Region-Guided Latent Reuse" (evidence region inside active region inside context
 * region; z = W*z_target + (1-W)*z_hist with W = 1 on the evidence region, 1 - smoothstep(d_hat) on the
 * transition band, 0 outside the active region) and "Joint Reuse in Intermediate Layers" (historical
 * connectivity kept only for active queries and their context tokens; tokens outside the active region
 * keep their cached computation); Appendix "Reuse-Scope Implementation Details" (dilation by 2 tokens,
 * then by a further 3, per latent frame on the H x W grid; Chebyshev distance to the evidence region
 * normalised by the largest distance attained in the band).
 *
 * carnator_build_regions:  evidence uint8 [T,Hg,Wg] (non-zero = member) -> active, context uint8 [T,Hg,Wg]
 *   and W fp32 [T,Hg,Wg]; r_active >= 1, r_context >= 0, r_active + r_context <= 32; the grid comes from
 *   `shape` (only T, Hg, Wg are read).  ws >= carnator_regions_workspace_bytes, 256-byte aligned.
 * carnator_fuse_latents:   z_out = W*z_target + (1-W)*z_hist over [channels, tokens] row-major tensors of
 *   `dtype` (CARNATOR_DTYPE_*), W fp32 [tokens]; tokens must be a multiple of 16 bytes worth of elements;
 *   z_out may alias z_target or z_hist.
 * carnator_region_block_flags: flags[i] = 1 iff block i of the token order (text first, then the grid,
 *   `block` tokens per block) holds a region token; text tokens count as members iff text_value != 0.
 * carnator_sparse_attn_region: as carnator_sparse_attn, with the evaluated pairs restricted to
 *   mask[b,h,I,J] != 0 && active_q[b,I] != 0 && context_k[b,J] != 0; query blocks with active_q == 0 are
 *   skipped: their rows of O and LSE are left untouched (the caller keeps the cached values there).
 *   active_q uint8 [B,nqb], context_k uint8 [B,nkb], both required.
 * All pointers are device pointers.
 * ------------------------------------------------------------------------ */
enum { CARNATOR_DTYPE_F32 = 0, CARNATOR_DTYPE_BF16 = 1 };

size_t carnator_regions_workspace_bytes(const carnator_shape* shape);

carnator_status carnator_build_regions(const uint8_t* evidence, const carnator_shape* shape,
                                       int32_t r_active, int32_t r_context,
                                       uint8_t* active, uint8_t* context, float* W,
                                       void* ws, size_t ws_bytes, void* stream);

carnator_status carnator_fuse_latents(const void* z_target, const void* z_hist, const float* W,
                                      int64_t channels, int64_t tokens, int32_t dtype,
                                      void* z_out, void* stream);

carnator_status carnator_region_block_flags(const uint8_t* region, const carnator_shape* shape,
                                            int32_t block, int32_t text_value,
                                            uint8_t* flags, void* stream);

carnator_status carnator_sparse_attn_region(const void* Q, const void* K, const void* V,
                                            const uint8_t* mask, const uint8_t* active_q, const uint8_t* context_k,
                                            const carnator_shape* shape,
                                            void* O, float* LSE,
                                            void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Seeded self-attention expansion (Early-Signature localisation).
 *
 * Paper: Section 3.2 and Appendix "Evidence Region Construction" -- noun and background seed token sets
 * I+ and I- are propagated through self-attention into the contrast score
 *   S_i = Agg_h [ max_{u in I+} A_h[i,u] - max_{u in I-} A_h[i,u] ],   A_h[i,u] = exp(s_iu - LSE_i),
 * A the dense self-attention weights.  Agg_h is taken as the mean over heads.  LSE is what a dense run of
 * carnator_sparse_attn (all-ones mask) returns for the same Q and K.
 *
 *   Q, K      device, bf16, strides of `shape`;  LSE device, fp32 [B,H,N]
 *   seeds     device, int32 [n_pos + n_neg] token indices in [0, N), positive set first, shared by all
 *             heads and batch entries; an empty set contributes 0
 *   per_head_opt  device, fp32 [B,H,N] or NULL: the per-head contrasts
 *   contrast  device, fp32 [B,N], written
 *   ws        device workspace, 256-byte aligned, >= carnator_seed_workspace_bytes (status header, the
 *             per-head contrasts, and the seed tokens' key rows gathered per head: 512 rows)
 *
 * Up to 512 seeds in all (and a query tensor that is not shared over heads or batch entries) run on the
 * tcgen05 tensor cores: a gather kernel, a persistent product-and-maximum kernel with bounded waits whose
 * status carnator_query_status(ws) returns, and the mean over heads.  Larger seed sets run on an mma.sync
 * kernel that streams the seed rows in chunks of 64.  A seed index outside [0, N) counts as a zero key row.
 * ------------------------------------------------------------------------ */
size_t carnator_seed_workspace_bytes(const carnator_shape* shape);

carnator_status carnator_seed_expansion(const void* Q, const void* K, const float* LSE,
                                        const int32_t* seeds, int32_t n_pos, int32_t n_neg,
                                        const carnator_shape* shape,
                                        float* per_head_opt, float* contrast,
                                        void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Host-side scalars of the reuse-validity gate and of its offline risk certificate.  No GPU work; all
 * pointers are HOST pointers; invalid arguments give NaN (0 for the gate).
 *
 * Paper: Section 3.2 -- d_size = |log(A_q / A_j)|, d_shape = 1 - Dice of the bounding-box-normalised object
 * indicators, d_context / d_color = CIEDE2000 difference of mean CIELAB colours, gate
 * g_tau = prod_k 1[d_k <= tau_k] over the applicable dimensions; Appendix "Risk-Aware Compatibility
 * Decision" -- one-sided Clopper-Pearson upper bound U_alpha(u, n) on the unsafe-reuse rate.
 *
 *   carnator_delta_e00            lab_a, lab_b: 3 doubles each (L*, a*, b*); k_L = k_C = k_H = 1
 *   carnator_context_discrepancy  d_context = max over the n_shared shared nouns of the CIEDE2000 difference between
 *                                 labs_q[3*o..3*o+2] and labs_j[3*o..3*o+2]; 0 when n_shared == 0
 *   carnator_size_discrepancy     positive tail-slice areas
 *   carnator_shape_discrepancy    binary indicators m_q [hq,wq], m_j [hj,wj]: each is cropped to its tight
 *                                 support box and resampled (cell centres, nearest) to resolution x resolution
 *   carnator_compatibility_gate   n dimensions; applicable may be NULL (= all); returns 1 iff all pass
 *   carnator_clopper_pearson_upper  unsafe u of accepted n at one-sided level alpha: the p solving
 *                                 P[Bin(n, p) <= u] = alpha (1 when u = n)
 * ------------------------------------------------------------------------ */
double  carnator_delta_e00(const double* lab_a, const double* lab_b);
double  carnator_context_discrepancy(const double* labs_q, const double* labs_j, int32_t n_shared);
double  carnator_size_discrepancy(double area_q, double area_j);
double  carnator_shape_discrepancy(const uint8_t* m_q, int32_t hq, int32_t wq,
                                   const uint8_t* m_j, int32_t hj, int32_t wj, int32_t resolution);
int32_t carnator_compatibility_gate(const double* d, const double* tau, const uint8_t* applicable, int32_t n);
double  carnator_clopper_pearson_upper(int32_t unsafe, int32_t accepted, double alpha);

/* ------------------------------------------------------------------------
 * carnator_sparse_attn_static -- carnator_sparse_attn for callers that cannot provide a workspace.
 *
 * (The paper has no counterpart for this call; it exists for deployment reasons only.)
 *
 * Some callers are not allowed to obtain device memory at the point where they call into this
 * library: code running under a memory budget that was fixed at start-up, plugins whose host
 * framework owns the allocator, and real-time loops in which cudaMalloc's implicit device
 * synchronisation is not acceptable.  They still own their inputs and outputs, but have nowhere
 * to put the compacted lists.  This form keeps that scratch in a fixed array that is part of the
 * library image itself: CARNATOR_STATIC_SCRATCH_BYTES of device memory, reserved on every GPU
 * the process uses the library on, from load until exit.
 *
 *   - Same arguments and results as carnator_sparse_attn, minus the workspace.
 *   - The call allocates and frees nothing, on the device or through any library.
 *   - A shape whose carnator_attn_workspace_bytes exceeds CARNATOR_STATIC_SCRATCH_BYTES is
 *     rejected with CARNATOR_ERR_WORKSPACE before anything is launched;
 *     carnator_last_cuda_error() then names both sizes.  (8 MiB covers e.g. B*H*nqb*nkb up to
 *     about two million block pairs: the Wan-1.3B-shaped layer fits, the 14B-shaped one does not.)
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current) and configures the kernels; make that first call outside of any
 *     stream capture.
 *   - All calls on one device share the one array.  It still holds the previous call's lists;
 *     each call clears the header it relies on and rewrites every list entry it reads, so
 *     back-to-back calls on one stream are safe.  Two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) race on the array: order them.
 *   - The device status word of this form lives at the start of the array.
 *     carnator_static_status(stream) is carnator_query_status for it: it synchronises `stream`,
 *     returns what kernels of earlier static-form calls on the current device reported
 *     (CARNATOR_OK, CARNATOR_ERR_DEVICE_TIMEOUT or CARNATOR_ERR_DEVICE_CHECK) and clears the word.
 *     It allocates nothing either.
 * ------------------------------------------------------------------------ */
#define CARNATOR_STATIC_SCRATCH_BYTES (8u << 20)

carnator_status carnator_sparse_attn_static(const void* Q, const void* K, const void* V,
                                            const uint8_t* mask, const uint8_t* recompute_rows,
                                            const carnator_shape* shape,
                                            void* O, float* LSE, void* stream);

carnator_status carnator_static_status(void* stream);

/* ------------------------------------------------------------------------
 * Status and diagnostics.
 * carnator_query_status synchronises `stream` and returns the status word that
 * kernels of earlier calls on this workspace may have set (CARNATOR_OK,
 * CARNATOR_ERR_DEVICE_TIMEOUT or CARNATOR_ERR_DEVICE_CHECK), then clears it.  The
 * word is initialised by the calls that take the workspace (build, compact, the
 * combined attention calls); querying a workspace no such call has used yet
 * returns whatever the memory held.  CARNATOR_ERR_DEVICE_CHECK is raised by the
 * tcgen05 attention kernel when a compacted list holds a key-block index outside
 * [0, nkb) or is not strictly ascending (only possible if the workspace was
 * modified between compaction and attention); the kernel then stops that query
 * block before loading anything.
 * carnator_kernel_launches returns how many kernels this library has launched in
 * the calling process so far (monotone counter).
 * ------------------------------------------------------------------------ */
carnator_status carnator_query_status(void* ws, void* stream);
/* Every wait inside a kernel of this library is bounded: after 2 s (less if the first 256 bytes of the workspace, the
 * header, carry a shorter wait_limit_ns at byte offset 40 -- written by tests only, the calls that take a workspace
 * reset it to 0 = default) the waiting role records CARNATOR_ERR_DEVICE_TIMEOUT, the CTA drains what it has in
 * flight, frees its tensor memory and returns; the device stays usable.
 * carnator_selftest_wait_timeout runs the wait helper on a barrier that is never armed (one warp, `limit_ns` between
 * 1 and 2e9): carnator_query_status(ws) must then report CARNATOR_ERR_DEVICE_TIMEOUT.  ws: device, >= 256 bytes,
 * 256-byte aligned. */
carnator_status carnator_selftest_wait_timeout(void* ws, uint64_t limit_ns, void* stream);

/* Testing aid: which path carnator_build_connectivity takes in top-k mode.  0 = by size (the default), 1 = always
 * the three separate kernels (pool, score, select), 2 = the persistent fused kernel wherever it supports the shape.
 * Both compute the same pooled scores up to the order of the fp32 sums.  Process-wide. */
void            carnator_debug_set_builder_path(int32_t path);
const char*     carnator_status_string(carnator_status s);
const char*     carnator_last_cuda_error(void);
int64_t         carnator_kernel_launches(void);
int32_t         carnator_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CARNATOR_H_ */
