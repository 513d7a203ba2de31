// C-ABI entry points of libcarnator: argument validation, workspace layout, kernel launches.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "carnator.h"
#include "common.cuh"
#include "builder.cuh"
#include "compact.cuh"
#include "attn_portable.cuh"
#include "attn_tcgen05.cuh"
#include "builder_fused.cuh"
#include "block_mass_tcgen05.cuh"
#include "regions.cuh"
#include "seed_expand.cuh"
#include "seed_expand_tcgen05.cuh"
#include "compat_host.inl"

using namespace carnator;

namespace {

std::atomic<long long> g_launches{0};
thread_local char g_cuda_error[256] = "";

carnator_status cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
    return CARNATOR_ERR_CUDA;
}

#define CUDA_TRY(expr)                                              \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr);       \
    } while (0)

#define LAUNCH_CHECK(name)                                          \
    do {                                                            \
        g_launches.fetch_add(1, std::memory_order_relaxed);         \
        cudaError_t e__ = cudaGetLastError();                       \
        if (e__ != cudaSuccess) return cuda_fail(e__, name);        \
    } while (0)

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bool strides_ok(const int64_t s[3]) {
    return s[0] >= 0 && s[1] >= 0 && s[2] > 0 && s[0] % 8 == 0 && s[1] % 8 == 0 && s[2] % 8 == 0;
}

carnator_status check_shape(const carnator_shape* s, bool need_v_o) {
    if (!s) return CARNATOR_ERR_INVALID_ARG;
    if (s->B <= 0 || s->H <= 0 || s->N <= 0 || s->D <= 0) return CARNATOR_ERR_INVALID_ARG;
    if (s->n_text < 0 || s->T < 0 || s->Hg < 0 || s->Wg < 0) return CARNATOR_ERR_INVALID_ARG;
    if (int64_t(s->n_text) + int64_t(s->T) * s->Hg * s->Wg != int64_t(s->N)) return CARNATOR_ERR_INVALID_ARG;
    if (s->block_q <= 0 || s->block_k <= 0) return CARNATOR_ERR_INVALID_ARG;
    if (s->D != 64 && s->D != 128) return CARNATOR_ERR_UNSUPPORTED;
    if ((s->block_q != 64 && s->block_q != 128) || (s->block_k != 64 && s->block_k != 128)) return CARNATOR_ERR_UNSUPPORTED;
    if (!strides_ok(s->q_stride) || !strides_ok(s->k_stride)) return CARNATOR_ERR_INVALID_ARG;
    if (s->q_stride[2] < s->D || s->k_stride[2] < s->D) return CARNATOR_ERR_INVALID_ARG;
    if (need_v_o) {
        if (!strides_ok(s->v_stride) || !strides_ok(s->o_stride)) return CARNATOR_ERR_INVALID_ARG;
        if (s->v_stride[2] < s->D || s->o_stride[2] < s->D) return CARNATOR_ERR_INVALID_ARG;
    }
    if (s->attn_impl < CARNATOR_IMPL_AUTO || s->attn_impl > CARNATOR_IMPL_TCGEN05) return CARNATOR_ERR_INVALID_ARG;
    if (std::isnan(s->softmax_scale) || std::isinf(s->softmax_scale)) return CARNATOR_ERR_INVALID_ARG;
    return CARNATOR_OK;
}

carnator_status check_params(const carnator_build_params* p) {
    if (!p) return CARNATOR_ERR_INVALID_ARG;
    if (p->mode != CARNATOR_MODE_TOPK && p->mode != CARNATOR_MODE_CUMMASS) return CARNATOR_ERR_INVALID_ARG;
    if (p->mode == CARNATOR_MODE_TOPK && !(p->keep_ratio > 0.f && p->keep_ratio <= 1.f)) return CARNATOR_ERR_INVALID_ARG;
    if (p->mode == CARNATOR_MODE_CUMMASS && !(p->mass > 0.f && p->mass <= 1.f)) return CARNATOR_ERR_INVALID_ARG;
    if (p->window_frames < -1) return CARNATOR_ERR_INVALID_ARG;
    return CARNATOR_OK;
}

// The device must be sm_100 (the kernels are built for sm_100a only).
carnator_status check_device() {
    static thread_local int cached_dev = -1;
    static thread_local carnator_status cached = CARNATOR_OK;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { cudaGetLastError(); snprintf(g_cuda_error, sizeof(g_cuda_error), "cudaGetDevice: %s", cudaGetErrorString(e)); return CARNATOR_ERR_UNSUPPORTED; }
    if (dev == cached_dev) return cached;
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { cudaGetLastError(); return CARNATOR_ERR_UNSUPPORTED; }
    cached_dev = dev;
    cached = (major == 10) ? CARNATOR_OK : CARNATOR_ERR_UNSUPPORTED;
    return cached;
}

float effective_scale(const carnator_shape* s) {
    return s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf(float(s->D));
}

int next_pow2(int x) { int p = 1; while (p < x) p <<= 1; return p; }

int topk_count_host(float ratio, int n) {
    if (n <= 0) return 0;
    double x = double(ratio) * double(n) - 1e-6;
    int k = int(std::ceil(x));
    return k < 1 ? 1 : (k > n ? n : k);
}

template <typename K>
carnator_status allow_smem(K kernel, size_t bytes) {
    CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes)));
    return CARNATOR_OK;
}

}  // namespace

namespace {
// Testing aid: 0 = choose by size, 1 = always the three kernels (pool, score, select), 2 = the persistent kernel
// wherever it supports the shape; so that the two paths can be compared on any input.
std::atomic<int> g_builder_path{0};

carnator_status sm_count(int* out) {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev != cached_dev) {
        int n = 0;
        CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        cached_dev = dev; cached = n;
    }
    *out = cached;
    return CARNATOR_OK;
}

constexpr size_t kMaxDynamicSmem = 226 * 1024;     // 227 KiB per CTA less the kernels' static shared memory

template <int D, int NPL, int PST, int AST>
carnator_status launch_fused_r(const FusedArgs& fa, const CUtensorMap (&maps)[4], int nkb, int sms, cudaStream_t stream) {
    const size_t smem = FusedSmem<D, PST, AST>::bytes(nkb, fa.nkb_pad);
    carnator_status st = allow_smem(build_fused_kernel<D, NPL, PST, AST>, smem);
    if (st != CARNATOR_OK) return st;
    // the register hand-over inside the kernel (setmaxnreg) only completes if the CTA owns 256 x 40 + 512 x 96 registers
    cudaFuncAttributes attr;
    CUDA_TRY(cudaFuncGetAttributes(&attr, build_fused_kernel<D, NPL, PST, AST>));
    if (attr.numRegs * kFusedThreads < 256 * 40 + 512 * 96) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "build_fused_kernel was built with %d registers per thread: too few for its setmaxnreg split", attr.numRegs);
        return CARNATOR_ERR_UNSUPPORTED;
    }
    build_fused_kernel<D, NPL, PST, AST><<<sms, kFusedThreads, smem, stream>>>(maps[0], maps[1], maps[2], maps[3], fa);
    LAUNCH_CHECK("build_fused_kernel");
    return CARNATOR_OK;
}

// Shared-memory plan of the fused kernel: pooling ring slots x buffers of the key-block score operand.  Three and three
// where the score rows (which grow with the number of key blocks) leave the room; a long layer gives up a ring slot
// rather than the third operand buffer (its scoring, not its pooling, is what the kernel waits for).  0: nothing fits.
template <int D>
int fused_plan_d(int nkb) {
    const int pad = (nkb + 3) & ~3;
    if (FusedSmem<D, 3, 3>::bytes(nkb, pad) <= kMaxDynamicSmem) return 33;
    if (FusedSmem<D, 2, 3>::bytes(nkb, pad) <= kMaxDynamicSmem) return 23;
    return 0;
}
int fused_plan(int D, int nkb) { return D == 128 ? fused_plan_d<128>(nkb) : fused_plan_d<64>(nkb); }
bool fused_fits(int D, int nkb) { return fused_plan(D, nkb) != 0; }

// a warp of the selection group keeps the NPL keys of its row in registers
template <int D, int NPL>
carnator_status launch_fused_p(const FusedArgs& fa, const CUtensorMap (&maps)[4], int nkb, int sms, cudaStream_t stream) {
    switch (fused_plan_d<D>(nkb)) {
        case 33: return launch_fused_r<D, NPL, 3, 3>(fa, maps, nkb, sms, stream);
        case 23: return launch_fused_r<D, NPL, 2, 3>(fa, maps, nkb, sms, stream);
        default: return CARNATOR_ERR_UNSUPPORTED;
    }
}

template <int D>
carnator_status launch_fused_d(const FusedArgs& fa, const CUtensorMap (&maps)[4], int nkb, int sms, cudaStream_t stream) {
    if (nkb <= 32 * 8) return launch_fused_p<D, 8>(fa, maps, nkb, sms, stream);
    if (nkb <= 32 * 20) return launch_fused_p<D, 20>(fa, maps, nkb, sms, stream);
    return launch_fused_p<D, 32>(fa, maps, nkb, sms, stream);
}

carnator_status launch_fused_builder(const FusedArgs& fa, const CUtensorMap (&maps)[4], int D, int nkb, int sms, cudaStream_t stream) {
    return D == 128 ? launch_fused_d<128>(fa, maps, nkb, sms, stream) : launch_fused_d<64>(fa, maps, nkb, sms, stream);
}
}  // namespace

extern "C" void carnator_debug_set_builder_path(int32_t path) { g_builder_path.store(path == 1 || path == 2 ? path : 0); }

// ------------------------------------------------------------------------------------------------
// builder
// ------------------------------------------------------------------------------------------------
extern "C" size_t carnator_build_workspace_bytes(const carnator_shape* s, const carnator_build_params* p) {
    if (check_shape(s, false) != CARNATOR_OK || check_params(p) != CARNATOR_OK) return 0;
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    return build_ws_layout(nullptr, s->B, s->H, nqb, nkb, s->D).bytes;
}

extern "C" carnator_status carnator_build_connectivity(const void* Q, const void* K, const carnator_shape* s,
                                                       const carnator_build_params* p, uint8_t* mask,
                                                       float* pooled_scores_opt, void* ws, size_t ws_bytes,
                                                       void* stream_) {
    carnator_status st = check_shape(s, false);
    if (st != CARNATOR_OK) return st;
    st = check_params(p);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !mask) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16)) return CARNATOR_ERR_INVALID_ARG;
    if (pooled_scores_opt && !aligned(pooled_scores_opt, 16)) return CARNATOR_ERR_INVALID_ARG;
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    if (nkb > kMaxKeyBlocksBuilder) return CARNATOR_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    BuildWs w = build_ws_layout(ws, s->B, s->H, nqb, nkb, s->D);
    if (ws_bytes < w.bytes) return CARNATOR_ERR_WORKSPACE;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    float* scores = pooled_scores_opt ? pooled_scores_opt : w.scores;

    // header and the per-head pooled-block counters are contiguous: one clear
    CUDA_TRY(cudaMemsetAsync(w.hdr, 0, align256(sizeof(WsHeader)) + align256(size_t(s->B) * s->H * 4), stream));

    PoolArgs pa;
    pa.X[0] = static_cast<const __nv_bfloat16*>(Q);
    pa.X[1] = static_cast<const __nv_bfloat16*>(K);
    for (int i = 0; i < 3; ++i) { pa.stride[0][i] = s->q_stride[i]; pa.stride[1][i] = s->k_stride[i]; }
    pa.block[0] = s->block_q; pa.block[1] = s->block_k;
    pa.nb[0] = nqb; pa.nb[1] = nkb;
    pa.out[0] = w.qbar; pa.out[1] = w.kbar;
    pa.N = s->N; pa.H = s->H;
    SelectArgs sa;
    sa.scores = scores; sa.mask = mask;
    sa.nqb = nqb; sa.nkb = nkb; sa.npad = next_pow2(nkb); sa.H = s->H;
    sa.mode = p->mode; sa.keep_ratio = p->keep_ratio; sa.mass = p->mass;
    sa.count_includes_forced = p->count_includes_forced;
    sa.k_all = topk_count_host(p->keep_ratio, nkb);
    sa.values_are_mass = 0;
    sa.g.N = s->N; sa.g.n_text = s->n_text; sa.g.hw = s->Hg * s->Wg > 0 ? s->Hg * s->Wg : 1; sa.g.T = s->T;
    sa.g.bq = s->block_q; sa.g.bk = s->block_k; sa.g.window = p->window_frames; sa.g.text_dense = p->text_dense;

    // The persistent kernel pays off once its scoring items fill the machine (its last items run after the pooling has
    // ended); smaller layers take the three kernels.
    int sms = 0;
    st = sm_count(&sms);
    if (st != CARNATOR_OK) return st;
    const int choice = g_builder_path.load();
    const bool fused_able = p->mode == CARNATOR_MODE_TOPK && nkb <= 32 * 32 && tma_strides_ok(s, s->q_stride) && tma_strides_ok(s, s->k_stride) &&
                            fused_fits(s->D, nkb);
    const bool fused_pays = int64_t(s->B) * s->H * ceil_div(nqb, kFusedRows) >= int64_t(sms);
    if (fused_able && (choice == 2 || (choice == 0 && fused_pays))) {
        // one persistent kernel: pooling, pooled scores and selection; the scores stay on chip
        FusedArgs fa;
        fa.pool = pa; fa.sel = sa;
        fa.scores_out = pooled_scores_opt; fa.done = w.done; fa.hdr = w.hdr;
        fa.split[0] = w.qsplit; fa.split[1] = w.ksplit;
        fa.B = s->B; fa.scale = effective_scale(s);
        fa.nkb_pad = (nkb + 3) & ~3;
        CUtensorMap maps[4];     // Q, K: one box = one block of tokens, all of D (rows >= N read as zero); the three-term
                                 // means of Q: one item's rows per box; of K: 128 rows x 32 columns per box
        const int64_t bh = int64_t(s->B) * s->H;
        const int pb = s->D == 64 ? 2 : 1;       // at D = 64 a pooling item is two consecutive blocks (one box)
        if (!tc::make_map_halves(&maps[0], Q, s->B, s->H, s->N, s->D, s->q_stride, pb * s->block_q) ||
            !tc::make_map_halves(&maps[1], K, s->B, s->H, s->N, s->D, s->k_stride, pb * s->block_k) ||
            !tc::make_map_2d(&maps[2], w.qsplit, 3 * bh * nqb, s->D, kFusedRows) ||
            !tc::make_map_2d(&maps[3], w.ksplit, 3 * bh * nkb, s->D, 128, 32)) {
            snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed or is unavailable");
            return CARNATOR_ERR_CUDA;
        }
        return launch_fused_builder(fa, maps, s->D, nkb, sms, stream);
    }
    // M1
    {
        dim3 grid(nqb > nkb ? nqb : nkb, s->H, 2 * s->B);
        if (s->D == 128) pool_kernel<128><<<grid, 256, 0, stream>>>(pa);
        else pool_kernel<64><<<grid, 256, 0, stream>>>(pa);
        LAUNCH_CHECK("pool_kernel");
    }
    // M2
    {
        dim3 grid(ceil_div(nkb, 64), ceil_div(nqb, 64), s->B * s->H);
        const float scale = effective_scale(s);
        if (s->D == 128) score_kernel<128><<<grid, 256, 0, stream>>>(w.qbar, w.kbar, scores, nqb, nkb, scale);
        else score_kernel<64><<<grid, 256, 0, stream>>>(w.qbar, w.kbar, scores, nqb, nkb, scale);
        LAUNCH_CHECK("score_kernel");
    }
    // M3
    {
        if (p->mode == CARNATOR_MODE_TOPK) {
            // register-resident selection, one warp per row
            const int rows = s->B * s->H * nqb;
            const int grid = ceil_div(rows, 8);
            const size_t tbl = size_t(nkb) * sizeof(int2);     // key-block frame table (<= 32 KiB)
            if (nkb <= 32 * 8) select_topk_kernel<8><<<grid, 256, tbl, stream>>>(sa, rows);
            else if (nkb <= 32 * 20) select_topk_kernel<20><<<grid, 256, tbl, stream>>>(sa, rows);
            else if (nkb <= 32 * 32) select_topk_kernel<32><<<grid, 256, tbl, stream>>>(sa, rows);
            else select_topk_kernel<128><<<grid, 256, tbl, stream>>>(sa, rows);
        } else {
            // cumulative-mass mode needs the sorted order: shared-memory bitonic sort, one CTA per row
            size_t smem = size_t(sa.npad) * 8 * 2 + ((nkb + 15) & ~15);
            st = allow_smem(select_kernel, 72 * 1024);
            if (st != CARNATOR_OK) return st;
            dim3 grid(nqb, s->H, s->B);
            select_kernel<<<grid, 256, smem, stream>>>(sa);
        }
        LAUNCH_CHECK("select_kernel");
    }
    return CARNATOR_OK;
}

// ------------------------------------------------------------------------------------------------
// exact block-mass builder
// ------------------------------------------------------------------------------------------------
namespace {
struct ExactWs { WsHeader* hdr; float* mass; size_t bytes; };
ExactWs exact_ws_layout(void* base, int B, int H, int nqb, int nkb) {
    ExactWs w;
    char* p = static_cast<char*>(base);
    w.hdr = reinterpret_cast<WsHeader*>(p);
    w.mass = reinterpret_cast<float*>(p + align256(sizeof(WsHeader)));
    w.bytes = align256(sizeof(WsHeader)) + align256(size_t(B) * H * nqb * size_t(nkb) * 4);
    return w;
}
}  // namespace

extern "C" size_t carnator_exact_workspace_bytes(const carnator_shape* s) {
    if (check_shape(s, false) != CARNATOR_OK) return 0;
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    return exact_ws_layout(nullptr, s->B, s->H, nqb, nkb).bytes;
}

extern "C" carnator_status carnator_build_connectivity_exact(const void* Q, const void* K, const float* LSE,
                                                             const carnator_shape* s, const carnator_build_params* p,
                                                             uint8_t* mask, float* block_mass_opt, void* ws,
                                                             size_t ws_bytes, void* stream_) {
    carnator_status st = check_shape(s, false);
    if (st != CARNATOR_OK) return st;
    if (!p) return CARNATOR_ERR_INVALID_ARG;
    if (!(p->mass > 0.f && p->mass <= 1.f) || p->window_frames < -1) return CARNATOR_ERR_INVALID_ARG;
    if (!Q || !K || !LSE || !mask) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(LSE, 4)) return CARNATOR_ERR_INVALID_ARG;
    if (block_mass_opt && !aligned(block_mass_opt, 4)) return CARNATOR_ERR_INVALID_ARG;
    if (s->block_q != tc::kBlock || s->block_k != tc::kBlock) return CARNATOR_ERR_UNSUPPORTED;
    if (!tma_strides_ok(s, s->q_stride) || !tma_strides_ok(s, s->k_stride)) return CARNATOR_ERR_UNSUPPORTED;   // read through TMA
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    if (nkb > kMaxKeyBlocksBuilder) return CARNATOR_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    ExactWs w = exact_ws_layout(ws, s->B, s->H, nqb, nkb);
    if (ws_bytes < w.bytes) return CARNATOR_ERR_WORKSPACE;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    float* mass = block_mass_opt ? block_mass_opt : w.mass;
    CUDA_TRY(cudaMemsetAsync(w.hdr, 0, sizeof(WsHeader), stream));

    tc::MassArgs ma;
    ma.LSE = LSE; ma.mass = mass; ma.hdr = w.hdr;
    ma.B = s->B; ma.H = s->H; ma.N = s->N; ma.nqb = nqb; ma.nkb = nkb;
    ma.scale_log2 = effective_scale(s) * kLog2e;
    st = launch_block_mass(Q, K, s->q_stride, s->k_stride, ma, s->D, stream, g_cuda_error, sizeof(g_cuda_error));
    if (st != CARNATOR_OK) return st;
    g_launches.fetch_add(1, std::memory_order_relaxed);

    SelectArgs sa;
    sa.scores = mass; sa.mask = mask;
    sa.nqb = nqb; sa.nkb = nkb; sa.npad = next_pow2(nkb); sa.H = s->H;
    sa.mode = CARNATOR_MODE_CUMMASS; sa.keep_ratio = 1.f; sa.mass = p->mass;
    sa.count_includes_forced = 1; sa.k_all = nkb; sa.values_are_mass = 1;
    sa.g.N = s->N; sa.g.n_text = s->n_text; sa.g.hw = s->Hg * s->Wg > 0 ? s->Hg * s->Wg : 1; sa.g.T = s->T;
    sa.g.bq = s->block_q; sa.g.bk = s->block_k; sa.g.window = p->window_frames; sa.g.text_dense = p->text_dense;
    const size_t smem = size_t(sa.npad) * 8 * 2 + ((nkb + 15) & ~15);
    st = allow_smem(select_kernel, 72 * 1024);
    if (st != CARNATOR_OK) return st;
    dim3 grid(nqb, s->H, s->B);
    select_kernel<<<grid, 256, smem, stream>>>(sa);
    LAUNCH_CHECK("select_kernel");
    return CARNATOR_OK;
}

// ------------------------------------------------------------------------------------------------
// compaction + attention
// ------------------------------------------------------------------------------------------------
extern "C" size_t carnator_attn_workspace_bytes(const carnator_shape* s) {
    if (check_shape(s, true) != CARNATOR_OK) return 0;
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    return attn_ws_layout(nullptr, s->B, s->H, nqb, nkb).bytes;
}

static carnator_status attn_ws_check(const carnator_shape* s, void* ws, size_t ws_bytes, AttnWs* out) {
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    *out = attn_ws_layout(ws, s->B, s->H, nqb, nkb);
    if (ws_bytes < out->bytes) return CARNATOR_ERR_WORKSPACE;
    return CARNATOR_OK;
}

static carnator_status compact_impl(const uint8_t* mask, const uint8_t* recompute_rows, const uint8_t* active_q,
                                    const uint8_t* context_k, const carnator_shape* s, void* ws, size_t ws_bytes,
                                    void* stream_) {
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    if (!mask) return CARNATOR_ERR_INVALID_ARG;
    AttnWs w;
    st = attn_ws_check(s, ws, ws_bytes, &w);
    if (st != CARNATOR_OK) return st;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    if (nqb > 12000) return CARNATOR_ERR_UNSUPPORTED;   // order kernel keeps one head's counts in shared memory
    CUDA_TRY(cudaMemsetAsync(w.hdr, 0, sizeof(WsHeader), stream));
    const int rows = s->B * s->H * nqb;
    compact_rows_kernel<<<ceil_div(rows, 8), 256, 0, stream>>>(mask, recompute_rows, s->B, s->H, nqb, nkb, w.counts, w.lists,
                                                               active_q, context_k);
    LAUNCH_CHECK("compact_rows_kernel");
    order_rows_kernel<<<s->B * s->H, 256, size_t(nqb) * 4, stream>>>(w.counts, nqb, w.order, w.hdr);
    LAUNCH_CHECK("order_rows_kernel");
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_compact_mask(const uint8_t* mask, const uint8_t* recompute_rows,
                                                 const carnator_shape* s, void* ws, size_t ws_bytes, void* stream_) {
    return compact_impl(mask, recompute_rows, nullptr, nullptr, s, ws, ws_bytes, stream_);
}

template <int D, int BQ>
static carnator_status launch_portable(const AttnArgs& a, cudaStream_t stream) {
    using C = PortableCfg<D, BQ>;
    carnator_status st = allow_smem(attn_portable_kernel<D, BQ>, C::smem_bytes);
    if (st != CARNATOR_OK) return st;
    dim3 grid(a.nqb, a.H, a.B);
    attn_portable_kernel<D, BQ><<<grid, C::NT, C::smem_bytes, stream>>>(a);
    LAUNCH_CHECK("attn_portable_kernel");
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_sparse_attn_compacted(const void* Q, const void* K, const void* V,
                                                          const carnator_shape* s, void* O, float* LSE,
                                                          void* ws, size_t ws_bytes, void* stream_) {
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !V || !O || !LSE) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(LSE, 4)) return CARNATOR_ERR_INVALID_ARG;
    AttnWs w;
    st = attn_ws_check(s, ws, ws_bytes, &w);
    if (st != CARNATOR_OK) return st;
    const bool tc_ok = tcgen05_supported(s);
    if (s->attn_impl == CARNATOR_IMPL_TCGEN05 && !tc_ok) return CARNATOR_ERR_UNSUPPORTED;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    AttnArgs a;
    a.Q = static_cast<const __nv_bfloat16*>(Q);
    a.K = static_cast<const __nv_bfloat16*>(K);
    a.V = static_cast<const __nv_bfloat16*>(V);
    a.O = static_cast<__nv_bfloat16*>(O);
    a.LSE = LSE;
    for (int i = 0; i < 3; ++i) { a.qs[i] = s->q_stride[i]; a.ks[i] = s->k_stride[i]; a.vs[i] = s->v_stride[i]; a.os[i] = s->o_stride[i]; }
    a.counts = w.counts; a.order = w.order; a.lists = w.lists; a.hdr = w.hdr;
    a.B = s->B; a.H = s->H; a.N = s->N;
    a.nqb = ceil_div(s->N, s->block_q); a.nkb = ceil_div(s->N, s->block_k);
    a.block_q = s->block_q; a.block_k = s->block_k;
    a.scale_log2 = effective_scale(s) * kLog2e;

    const bool use_tc = tc_ok && s->attn_impl != CARNATOR_IMPL_PORTABLE;
    if (use_tc) {
        long long n = 0;
        st = launch_tcgen05(a, s, stream, g_cuda_error, sizeof(g_cuda_error), &n);
        g_launches.fetch_add(n, std::memory_order_relaxed);
        return st;
    }
    if (s->D == 128 && s->block_q == 128) return launch_portable<128, 128>(a, stream);
    if (s->D == 128 && s->block_q == 64) return launch_portable<128, 64>(a, stream);
    if (s->D == 64 && s->block_q == 128) return launch_portable<64, 128>(a, stream);
    return launch_portable<64, 64>(a, stream);
}

extern "C" carnator_status carnator_sparse_attn(const void* Q, const void* K, const void* V, const uint8_t* mask,
                                                const uint8_t* recompute_rows, const carnator_shape* s, void* O,
                                                float* LSE, void* ws, size_t ws_bytes, void* stream) {
    // validate everything before the first launch
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !V || !O || !LSE || !mask) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(LSE, 4)) return CARNATOR_ERR_INVALID_ARG;
    if (s->attn_impl == CARNATOR_IMPL_TCGEN05 && !tcgen05_supported(s)) return CARNATOR_ERR_UNSUPPORTED;
    st = carnator_compact_mask(mask, recompute_rows, s, ws, ws_bytes, stream);
    if (st != CARNATOR_OK) return st;
    return carnator_sparse_attn_compacted(Q, K, V, s, O, LSE, ws, ws_bytes, stream);
}

extern "C" carnator_status carnator_compacted_tiles(const carnator_shape* s, const void* ws, size_t ws_bytes,
                                                    void* stream_, int64_t* tiles) {
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    if (!tiles) return CARNATOR_ERR_INVALID_ARG;
    AttnWs w;
    st = attn_ws_check(s, const_cast<void*>(ws), ws_bytes, &w);
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    WsHeader h;
    CUDA_TRY(cudaMemcpyAsync(&h, w.hdr, sizeof(WsHeader), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    *tiles = int64_t(h.tiles);
    return CARNATOR_OK;
}

// ------------------------------------------------------------------------------------------------
// host-buffer forms
// ------------------------------------------------------------------------------------------------
namespace {
// The host-buffer attention call works through the heads in chunks, so that the copy-in of chunk k+1, the kernels of
// chunk k and the copy-out of chunk k-1 overlap (PCIe is full duplex and the copy engines run beside the SMs).
constexpr int kMaxHostChunks = 64;
constexpr size_t kHostChunkBytes = size_t(64) << 20;     // target size of one tensor's share of a chunk

struct HostChunks {
    int heads;          // heads per chunk (the last chunk of a batch entry may be shorter)
    int per_batch;      // chunks per batch entry
    int count;          // per_batch * B
};
HostChunks host_chunks(const carnator_shape* s) {
    const size_t per_head = size_t(s->N) * s->D * 2;
    int hc = int(std::min<size_t>(size_t(s->H), std::max<size_t>(1, (kHostChunkBytes + per_head - 1) / per_head)));
    while (int64_t(s->B) * ceil_div(s->H, hc) > kMaxHostChunks && hc < s->H) ++hc;
    HostChunks c;
    c.heads = hc;
    c.per_batch = ceil_div(s->H, hc);
    c.count = c.per_batch * s->B;
    return c;
}

struct HostArena {
    char *Q, *K, *V, *O;
    float* LSE;
    uint8_t *mask, *rec;
    char* ws;                   // one workspace per chunk, ws_stride apart
    size_t ws_stride, bytes;
    HostChunks chunks;
};
HostArena attn_arena_layout(void* base, const carnator_shape* s) {
    HostArena a;
    char* p = static_cast<char*>(base);
    const int nqb = ceil_div(s->N, s->block_q), nkb = ceil_div(s->N, s->block_k);
    const size_t t = align256(size_t(s->B) * s->H * s->N * s->D * 2);
    size_t off = 0;
    a.Q = p + off; off += t;
    a.K = p + off; off += t;
    a.V = p + off; off += t;
    a.O = p + off; off += t;
    a.LSE = reinterpret_cast<float*>(p + off); off += align256(size_t(s->B) * s->H * s->N * 4);
    a.mask = reinterpret_cast<uint8_t*>(p + off); off += align256(size_t(s->B) * s->H * nqb * nkb);
    a.rec = reinterpret_cast<uint8_t*>(p + off); off += align256(size_t(s->B) * nqb);
    a.chunks = host_chunks(s);
    a.ws = p + off;
    a.ws_stride = align256(attn_ws_layout(nullptr, 1, a.chunks.heads, nqb, nkb).bytes);
    off += a.ws_stride * a.chunks.count;
    a.bytes = off;
    return a;
}
void contiguous_strides(carnator_shape* c) {
    const int64_t n = c->N, d = c->D, h = c->H;
    int64_t st[3] = {h * n * d, n * d, d};
    for (int i = 0; i < 3; ++i) c->q_stride[i] = c->k_stride[i] = c->v_stride[i] = c->o_stride[i] = st[i];
}

// Streams and events of the chunk pipeline: made once per device and kept.  One host-buffer attention call at a time
// uses them (g_pipe_mu is held for the whole call).
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    cudaEvent_t ev_in[kMaxHostChunks], ev_comp[kMaxHostChunks];
};
constexpr int kMaxPipeDevices = 32;
std::mutex g_pipe_mu;
HostPipe g_pipes[kMaxPipeDevices];

carnator_status get_pipe(HostPipe** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxPipeDevices) return CARNATOR_ERR_UNSUPPORTED;
    HostPipe& p = g_pipes[dev];
    if (!p.ready) {
        CUDA_TRY(cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking));
        CUDA_TRY(cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking));
        CUDA_TRY(cudaEventCreateWithFlags(&p.ev_start, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&p.ev_out, cudaEventDisableTiming));
        for (int k = 0; k < kMaxHostChunks; ++k) {
            CUDA_TRY(cudaEventCreateWithFlags(&p.ev_in[k], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&p.ev_comp[k], cudaEventDisableTiming));
        }
        p.ready = true;
    }
    *out = &p;
    return CARNATOR_OK;
}

// The body of the pipelined call; the caller drains all three streams whatever this returns.
carnator_status attn_host_pipeline(const char* Q, const char* K, const char* V, const uint8_t* mask, const uint8_t* rec,
                                   const carnator_shape& s, char* O, float* LSE, const HostArena& a, HostPipe& pipe,
                                   cudaStream_t stream) {
    const int nqb = ceil_div(s.N, s.block_q), nkb = ceil_div(s.N, s.block_k);
    const size_t head_t = size_t(s.N) * s.D * 2, head_m = size_t(nqb) * nkb, head_l = size_t(s.N) * 4;
    // everything queued on the caller's stream so far comes first
    CUDA_TRY(cudaEventRecord(pipe.ev_start, stream));
    CUDA_TRY(cudaStreamWaitEvent(pipe.s_in, pipe.ev_start, 0));
    CUDA_TRY(cudaStreamWaitEvent(pipe.s_out, pipe.ev_start, 0));
    if (rec) CUDA_TRY(cudaMemcpyAsync(a.rec, rec, size_t(s.B) * nqb, cudaMemcpyHostToDevice, pipe.s_in));
    int k = 0;
    for (int b = 0; b < s.B; ++b) {
        for (int h0 = 0; h0 < s.H; h0 += a.chunks.heads, ++k) {
            const int hc = std::min(a.chunks.heads, s.H - h0);
            const size_t first = size_t(b) * s.H + h0;
            const size_t ot = first * head_t, om = first * head_m, ol = first * head_l;
            CUDA_TRY(cudaMemcpyAsync(a.Q + ot, Q + ot, hc * head_t, cudaMemcpyHostToDevice, pipe.s_in));
            CUDA_TRY(cudaMemcpyAsync(a.K + ot, K + ot, hc * head_t, cudaMemcpyHostToDevice, pipe.s_in));
            CUDA_TRY(cudaMemcpyAsync(a.V + ot, V + ot, hc * head_t, cudaMemcpyHostToDevice, pipe.s_in));
            CUDA_TRY(cudaMemcpyAsync(a.mask + om, mask + om, hc * head_m, cudaMemcpyHostToDevice, pipe.s_in));
            CUDA_TRY(cudaEventRecord(pipe.ev_in[k], pipe.s_in));
            CUDA_TRY(cudaStreamWaitEvent(stream, pipe.ev_in[k], 0));
            carnator_shape c = s;             // one batch entry, hc heads, strides of the whole tensor
            c.B = 1;
            c.H = hc;
            carnator_status st = carnator_sparse_attn(a.Q + ot, a.K + ot, a.V + ot, a.mask + om, rec ? a.rec + size_t(b) * nqb : nullptr,
                                                      &c, a.O + ot, reinterpret_cast<float*>(reinterpret_cast<char*>(a.LSE) + ol),
                                                      a.ws + size_t(k) * a.ws_stride, a.ws_stride, stream);
            if (st != CARNATOR_OK) return st;
            CUDA_TRY(cudaEventRecord(pipe.ev_comp[k], stream));
            CUDA_TRY(cudaStreamWaitEvent(pipe.s_out, pipe.ev_comp[k], 0));
            CUDA_TRY(cudaMemcpyAsync(O + ot, a.O + ot, hc * head_t, cudaMemcpyDeviceToHost, pipe.s_out));
            CUDA_TRY(cudaMemcpyAsync(reinterpret_cast<char*>(LSE) + ol, reinterpret_cast<char*>(a.LSE) + ol, hc * head_l,
                                     cudaMemcpyDeviceToHost, pipe.s_out));
        }
    }
    CUDA_TRY(cudaEventRecord(pipe.ev_out, pipe.s_out));
    CUDA_TRY(cudaStreamWaitEvent(stream, pipe.ev_out, 0));
    return CARNATOR_OK;
}
}  // namespace

extern "C" size_t carnator_attn_host_arena_bytes(const carnator_shape* s_in) {
    if (!s_in) return 0;
    carnator_shape s = *s_in;
    contiguous_strides(&s);
    if (check_shape(&s, true) != CARNATOR_OK) return 0;
    return attn_arena_layout(nullptr, &s).bytes;
}

extern "C" carnator_status carnator_sparse_attn_host(const void* Q, const void* K, const void* V, const uint8_t* mask,
                                                     const uint8_t* recompute_rows, const carnator_shape* s_in,
                                                     void* O, float* LSE, void* arena, size_t arena_bytes,
                                                     void* stream_) {
    if (!s_in) return CARNATOR_ERR_INVALID_ARG;
    carnator_shape s = *s_in;
    contiguous_strides(&s);
    carnator_status st = check_shape(&s, true);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !V || !mask || !O || !LSE) return CARNATOR_ERR_INVALID_ARG;
    if (!arena || !aligned(arena, 256)) return CARNATOR_ERR_WORKSPACE;
    HostArena a = attn_arena_layout(arena, &s);
    if (arena_bytes < a.bytes) return CARNATOR_ERR_WORKSPACE;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::lock_guard<std::mutex> lock(g_pipe_mu);
    HostPipe* pipe = nullptr;
    st = get_pipe(&pipe);
    if (st != CARNATOR_OK) return st;
    st = attn_host_pipeline(static_cast<const char*>(Q), static_cast<const char*>(K), static_cast<const char*>(V), mask,
                            recompute_rows, s, static_cast<char*>(O), LSE, a, *pipe, stream);
    // nothing of this call may still be in flight when it returns, whatever happened above
    const cudaError_t e1 = cudaStreamSynchronize(pipe->s_in), e2 = cudaStreamSynchronize(stream), e3 = cudaStreamSynchronize(pipe->s_out);
    if (st != CARNATOR_OK) return st;
    if (e1 != cudaSuccess) return cuda_fail(e1, "cudaStreamSynchronize(copy-in stream)");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaStreamSynchronize(stream)");
    if (e3 != cudaSuccess) return cuda_fail(e3, "cudaStreamSynchronize(copy-out stream)");
    for (int k = 0; k < a.chunks.count; ++k) {         // every chunk has its own status header; report the first failure
        const carnator_status sk = carnator_query_status(a.ws + size_t(k) * a.ws_stride, stream_);
        if (sk != CARNATOR_OK && st == CARNATOR_OK) st = sk;
    }
    return st;
}

extern "C" size_t carnator_build_host_arena_bytes(const carnator_shape* s_in, const carnator_build_params* p) {
    if (!s_in) return 0;
    carnator_shape s = *s_in;
    contiguous_strides(&s);
    if (check_shape(&s, false) != CARNATOR_OK || check_params(p) != CARNATOR_OK) return 0;
    const int nqb = ceil_div(s.N, s.block_q), nkb = ceil_div(s.N, s.block_k);
    const size_t t = align256(size_t(s.B) * s.H * s.N * s.D * 2);
    return 2 * t + align256(size_t(s.B) * s.H * nqb * nkb) + build_ws_layout(nullptr, s.B, s.H, nqb, nkb, s.D).bytes;
}

extern "C" carnator_status carnator_build_connectivity_host(const void* Q, const void* K, const carnator_shape* s_in,
                                                            const carnator_build_params* p, uint8_t* mask,
                                                            void* arena, size_t arena_bytes, void* stream_) {
    if (!s_in) return CARNATOR_ERR_INVALID_ARG;
    carnator_shape s = *s_in;
    contiguous_strides(&s);
    carnator_status st = check_shape(&s, false);
    if (st != CARNATOR_OK) return st;
    st = check_params(p);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !mask) return CARNATOR_ERR_INVALID_ARG;
    if (!arena || !aligned(arena, 256)) return CARNATOR_ERR_WORKSPACE;
    const size_t need = carnator_build_host_arena_bytes(&s, p);
    if (arena_bytes < need) return CARNATOR_ERR_WORKSPACE;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int nqb = ceil_div(s.N, s.block_q), nkb = ceil_div(s.N, s.block_k);
    const size_t t = size_t(s.B) * s.H * s.N * s.D * 2, ta = align256(t);
    const size_t mbytes = size_t(s.B) * s.H * nqb * nkb;
    char* base = static_cast<char*>(arena);
    char* dQ = base;
    char* dK = base + ta;
    uint8_t* dM = reinterpret_cast<uint8_t*>(base + 2 * ta);
    void* ws = base + 2 * ta + align256(mbytes);
    const size_t ws_bytes = need - (2 * ta + align256(mbytes));
    CUDA_TRY(cudaMemcpyAsync(dQ, Q, t, cudaMemcpyHostToDevice, stream));
    CUDA_TRY(cudaMemcpyAsync(dK, K, t, cudaMemcpyHostToDevice, stream));
    st = carnator_build_connectivity(dQ, dK, &s, p, dM, nullptr, ws, ws_bytes, stream_);
    if (st != CARNATOR_OK) return st;
    CUDA_TRY(cudaMemcpyAsync(mask, dM, mbytes, cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return carnator_query_status(ws, stream_);
}

// ------------------------------------------------------------------------------------------------
// reuse regions, latent fusion, region-restricted attention
// ------------------------------------------------------------------------------------------------
extern "C" size_t carnator_regions_workspace_bytes(const carnator_shape* s) {
    if (!s || s->T <= 0 || s->Hg <= 0 || s->Wg <= 0) return 0;
    return align256(sizeof(WsHeader)) + align256(size_t(s->T) * s->Hg * s->Wg);
}

extern "C" carnator_status carnator_build_regions(const uint8_t* evidence, const carnator_shape* s, int32_t r_active,
                                                  int32_t r_context, uint8_t* active, uint8_t* context, float* W,
                                                  void* ws, size_t ws_bytes, void* stream_) {
    if (!s || s->T <= 0 || s->Hg <= 0 || s->Wg <= 0) return CARNATOR_ERR_INVALID_ARG;
    if (!evidence || !active || !context || !W) return CARNATOR_ERR_INVALID_ARG;
    if (r_active < 1 || r_context < 0 || r_active + r_context > 32) return CARNATOR_ERR_INVALID_ARG;
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    if (ws_bytes < carnator_regions_workspace_bytes(s)) return CARNATOR_ERR_WORKSPACE;
    carnator_status st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    WsHeader* hdr = static_cast<WsHeader*>(ws);
    uint8_t* dist = static_cast<uint8_t*>(ws) + align256(sizeof(WsHeader));
    const int n = s->T * s->Hg * s->Wg;
    CUDA_TRY(cudaMemsetAsync(hdr, 0, sizeof(WsHeader), stream));
    region_distance_kernel<<<ceil_div(n, 256), 256, 0, stream>>>(evidence, s->T, s->Hg, s->Wg, r_active, r_context, dist,
                                                                 active, context, hdr);
    LAUNCH_CHECK("region_distance_kernel");
    region_weight_kernel<<<ceil_div(n, 256), 256, 0, stream>>>(dist, n, r_active, hdr, W);
    LAUNCH_CHECK("region_weight_kernel");
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_fuse_latents(const void* z_target, const void* z_hist, const float* W,
                                                 int64_t channels, int64_t tokens, int32_t dtype, void* z_out,
                                                 void* stream_) {
    if (!z_target || !z_hist || !W || !z_out || channels <= 0 || tokens <= 0) return CARNATOR_ERR_INVALID_ARG;
    if (dtype != CARNATOR_DTYPE_F32 && dtype != CARNATOR_DTYPE_BF16) return CARNATOR_ERR_INVALID_ARG;
    const int vec = dtype == CARNATOR_DTYPE_F32 ? 4 : 8;
    if (tokens % vec != 0) return CARNATOR_ERR_UNSUPPORTED;          // rows of 16 bytes
    if (!aligned(z_target, 16) || !aligned(z_hist, 16) || !aligned(z_out, 16) || !aligned(W, 4)) return CARNATOR_ERR_INVALID_ARG;
    carnator_status st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t work = channels * (tokens / vec);
    const unsigned grid = unsigned((work + 255) / 256);
    if (dtype == CARNATOR_DTYPE_F32)
        fuse_latents_kernel<float, 4><<<grid, 256, 0, stream>>>(static_cast<const float*>(z_target), static_cast<const float*>(z_hist),
                                                               W, channels, tokens, static_cast<float*>(z_out));
    else
        fuse_latents_kernel<__nv_bfloat16, 8><<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(z_target),
                                                                       static_cast<const __nv_bfloat16*>(z_hist), W, channels,
                                                                       tokens, static_cast<__nv_bfloat16*>(z_out));
    LAUNCH_CHECK("fuse_latents_kernel");
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_region_block_flags(const uint8_t* region, const carnator_shape* s, int32_t block,
                                                       int32_t text_value, uint8_t* flags, void* stream_) {
    if (!s || !region || !flags || block <= 0) return CARNATOR_ERR_INVALID_ARG;
    if (s->n_text < 0 || s->T <= 0 || s->Hg <= 0 || s->Wg <= 0) return CARNATOR_ERR_INVALID_ARG;
    carnator_status st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int n_video = s->T * s->Hg * s->Wg;
    const int nblocks = ceil_div(s->n_text + n_video, block);
    region_block_flags_kernel<<<ceil_div(nblocks, 8), 256, 0, stream>>>(region, s->n_text, n_video, block, text_value, nblocks, flags);
    LAUNCH_CHECK("region_block_flags_kernel");
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_sparse_attn_region(const void* Q, const void* K, const void* V, const uint8_t* mask,
                                                       const uint8_t* active_q, const uint8_t* context_k,
                                                       const carnator_shape* s, void* O, float* LSE, void* ws,
                                                       size_t ws_bytes, void* stream) {
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !V || !O || !LSE || !mask || !active_q || !context_k) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(LSE, 4)) return CARNATOR_ERR_INVALID_ARG;
    if (s->attn_impl == CARNATOR_IMPL_TCGEN05 && !tcgen05_supported(s)) return CARNATOR_ERR_UNSUPPORTED;
    st = compact_impl(mask, nullptr, active_q, context_k, s, ws, ws_bytes, stream);
    if (st != CARNATOR_OK) return st;
    return carnator_sparse_attn_compacted(Q, K, V, s, O, LSE, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------------
// seeded self-attention expansion
// ------------------------------------------------------------------------------------------------
extern "C" size_t carnator_seed_workspace_bytes(const carnator_shape* s) {
    if (check_shape(s, false) != CARNATOR_OK) return 0;
    // header | per-head contrasts [B,H,N] fp32 | gathered seed key rows [B,H,512,D] bf16
    return align256(sizeof(WsHeader)) + align256(size_t(s->B) * s->H * s->N * 4) + align256(seed_gather_bytes(s));
}

extern "C" carnator_status carnator_seed_expansion(const void* Q, const void* K, const float* LSE, const int32_t* seeds,
                                                   int32_t n_pos, int32_t n_neg, const carnator_shape* s,
                                                   float* per_head_opt, float* contrast, void* ws, size_t ws_bytes,
                                                   void* stream_) {
    carnator_status st = check_shape(s, false);
    if (st != CARNATOR_OK) return st;
    if (!Q || !K || !LSE || !contrast || n_pos < 0 || n_neg < 0 || (n_pos + n_neg > 0 && !seeds)) return CARNATOR_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16)) return CARNATOR_ERR_INVALID_ARG;
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    if (ws_bytes < carnator_seed_workspace_bytes(s)) return CARNATOR_ERR_WORKSPACE;
    st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    SeedArgs a;
    a.Q = static_cast<const __nv_bfloat16*>(Q); a.K = static_cast<const __nv_bfloat16*>(K);
    for (int i = 0; i < 3; ++i) { a.qs[i] = s->q_stride[i]; a.ks[i] = s->k_stride[i]; }
    a.LSE = LSE; a.seeds = seeds; a.n_pos = n_pos; a.n_neg = n_neg;
    a.per_head = per_head_opt ? per_head_opt : reinterpret_cast<float*>(static_cast<char*>(ws) + align256(sizeof(WsHeader)));
    a.B = s->B; a.H = s->H; a.N = s->N;
    a.scale_log2 = effective_scale(s) * kLog2e;
    const int64_t n_bn = int64_t(s->B) * s->N;
    if (seed_tcgen05_supported(s, n_pos + n_neg)) {
        WsHeader* hdr = static_cast<WsHeader*>(ws);
        CUDA_TRY(cudaMemsetAsync(hdr, 0, sizeof(WsHeader), stream));
        int sms = 0;
        st = sm_count(&sms);
        if (st != CARNATOR_OK) return st;
        tc::SeedGatherArgs ga;
        ga.K = a.K; for (int i = 0; i < 3; ++i) ga.ks[i] = a.ks[i];
        ga.seeds = seeds; ga.n_seeds = n_pos + n_neg; ga.H = s->H; ga.N = s->N;
        ga.out = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + align256(sizeof(WsHeader)) +
                                                   align256(size_t(s->B) * s->H * s->N * 4));
        tc::SeedTcArgs ta;
        ta.LSE = LSE; ta.per_head = a.per_head; ta.hdr = hdr;
        ta.n_pos = n_pos; ta.n_seeds = n_pos + n_neg;
        ta.B = s->B; ta.H = s->H; ta.N = s->N; ta.nqb = ceil_div(s->N, tc::kBlock);
        ta.tiles = s->B * s->H * ta.nqb;
        ta.scale_log2 = a.scale_log2;
        CUtensorMap mq, ms;      // the gathered rows as one [B*H*512, D] array: a box = 256 seed rows x 64 elements
        if (!tc::make_map(&mq, Q, s->B, s->H, s->N, s->D, s->q_stride, tc::kBlock) ||
            !tc::make_map_2d(&ms, ga.out, int64_t(s->B) * s->H * tc::kSeedCap, s->D, tc::kSeedChunk)) {
            snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed or is unavailable");
            return CARNATOR_ERR_CUDA;
        }
        st = s->D == 128 ? launch_seed_tc<128>(ga, ta, mq, ms, sms, stream, g_cuda_error, sizeof(g_cuda_error))
                         : launch_seed_tc<64>(ga, ta, mq, ms, sms, stream, g_cuda_error, sizeof(g_cuda_error));
        if (st != CARNATOR_OK) return st;
        head_mean_kernel<<<unsigned((n_bn + 255) / 256), 256, 0, stream>>>(a.per_head, s->B, s->H, s->N, contrast);
        LAUNCH_CHECK("head_mean_kernel");
        return CARNATOR_OK;
    }
    dim3 grid(ceil_div(s->N, 128), s->H, s->B);
    if (s->D == 128) {
        const size_t smem = size_t(128 + 2 * 64) * (128 + 8) * 2;
        st = allow_smem(seed_expand_kernel<128>, smem);
        if (st != CARNATOR_OK) return st;
        seed_expand_kernel<128><<<grid, 256, smem, stream>>>(a);
    } else {
        const size_t smem = size_t(128 + 2 * 64) * (64 + 8) * 2;
        st = allow_smem(seed_expand_kernel<64>, smem);
        if (st != CARNATOR_OK) return st;
        seed_expand_kernel<64><<<grid, 256, smem, stream>>>(a);
    }
    LAUNCH_CHECK("seed_expand_kernel");
    const int64_t n = int64_t(s->B) * s->N;
    head_mean_kernel<<<unsigned((n + 255) / 256), 256, 0, stream>>>(a.per_head, s->B, s->H, s->N, contrast);
    LAUNCH_CHECK("head_mean_kernel");
    return CARNATOR_OK;
}

// ------------------------------------------------------------------------------------------------
// host-side compatibility scalars and risk bound
// ------------------------------------------------------------------------------------------------
extern "C" double carnator_delta_e00(const double* lab_a, const double* lab_b) {
    if (!lab_a || !lab_b) return NAN;
    return carnator_host::delta_e00(lab_a, lab_b);
}

extern "C" double carnator_context_discrepancy(const double* labs_q, const double* labs_j, int32_t n_shared) {
    if (n_shared < 0 || (n_shared > 0 && (!labs_q || !labs_j))) return NAN;
    double d = 0.0;                                        // no shared noun: the dimension reads 0
    for (int32_t o = 0; o < n_shared; ++o) d = std::max(d, carnator_host::delta_e00(labs_q + 3 * o, labs_j + 3 * o));
    return d;
}

extern "C" double carnator_size_discrepancy(double area_q, double area_j) {
    if (!(area_q > 0.0) || !(area_j > 0.0)) return NAN;
    return std::fabs(std::log(area_q / area_j));
}

extern "C" double carnator_shape_discrepancy(const uint8_t* m_q, int32_t hq, int32_t wq, const uint8_t* m_j, int32_t hj,
                                             int32_t wj, int32_t resolution) {
    if (!m_q || !m_j || hq <= 0 || wq <= 0 || hj <= 0 || wj <= 0 || resolution <= 0) return NAN;
    std::vector<uint8_t> a, b;
    if (!carnator_host::bbox_normalize(m_q, hq, wq, resolution, a) || !carnator_host::bbox_normalize(m_j, hj, wj, resolution, b)) return NAN;
    long inter = 0, na = 0, nb = 0;
    for (size_t i = 0; i < a.size(); ++i) { inter += a[i] & b[i]; na += a[i]; nb += b[i]; }
    return 1.0 - 2.0 * double(inter) / double(na + nb);
}

extern "C" int32_t carnator_compatibility_gate(const double* d, const double* tau, const uint8_t* applicable, int32_t n) {
    if (!d || !tau || n < 0) return 0;
    for (int k = 0; k < n; ++k)
        if ((!applicable || applicable[k]) && !(d[k] <= tau[k])) return 0;
    return 1;
}

extern "C" double carnator_clopper_pearson_upper(int32_t unsafe, int32_t accepted, double alpha) {
    if (accepted <= 0 || unsafe < 0 || unsafe > accepted || !(alpha > 0.0 && alpha < 1.0)) return NAN;
    return carnator_host::clopper_pearson_upper(unsafe, accepted, alpha);
}

// ------------------------------------------------------------------------------------------------
// static-scratch form: for callers that may not obtain device memory (fixed budgets, plugins whose host
// owns the allocator, loops that cannot tolerate cudaMalloc's synchronisation).  The scratch is a
// file-scope device array; in host code its name is only a handle, so the device address is looked up
// with cudaGetSymbolAddress once per device (under that device) and that pointer is what kernels get.
// ------------------------------------------------------------------------------------------------
namespace {
static __device__ __align__(256) unsigned char g_static_scratch[CARNATOR_STATIC_SCRATCH_BYTES];
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_mu;
}  // namespace

namespace {
// Device address of the built-in array on the current device (looked up once per device, with that device current).
carnator_status static_scratch_ptr(void** out) {
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CARNATOR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return CARNATOR_OK;
}
}  // namespace

extern "C" carnator_status carnator_sparse_attn_static(const void* Q, const void* K, const void* V,
                                                       const uint8_t* mask, const uint8_t* recompute_rows,
                                                       const carnator_shape* s, void* O, float* LSE, void* stream) {
    carnator_status st = check_shape(s, true);
    if (st != CARNATOR_OK) return st;
    const size_t need = carnator_attn_workspace_bytes(s);
    if (need == 0 || need > size_t(CARNATOR_STATIC_SCRATCH_BYTES)) {
        snprintf(g_cuda_error, sizeof(g_cuda_error),
                 "carnator_sparse_attn_static: this shape needs %zu bytes of scratch, the built-in array holds %zu",
                 need, size_t(CARNATOR_STATIC_SCRATCH_BYTES));
        return CARNATOR_ERR_WORKSPACE;
    }
    st = check_device();
    if (st != CARNATOR_OK) return st;
    void* scratch = nullptr;
    st = static_scratch_ptr(&scratch);
    if (st != CARNATOR_OK) return st;
    // carnator_sparse_attn clears the header and rewrites every list entry it later reads.
    return carnator_sparse_attn(Q, K, V, mask, recompute_rows, s, O, LSE, scratch, size_t(CARNATOR_STATIC_SCRATCH_BYTES), stream);
}

extern "C" carnator_status carnator_static_status(void* stream) {
    carnator_status st = check_device();
    if (st != CARNATOR_OK) return st;
    void* scratch = nullptr;
    st = static_scratch_ptr(&scratch);
    if (st != CARNATOR_OK) return st;
    return carnator_query_status(scratch, stream);       // the array starts with the same header as a workspace
}

// ------------------------------------------------------------------------------------------------
// status
// ------------------------------------------------------------------------------------------------
extern "C" carnator_status carnator_query_status(void* ws, void* stream_) {
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    WsHeader h;
    CUDA_TRY(cudaMemcpyAsync(&h, ws, sizeof(WsHeader), cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    if (h.status != 0) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "device status %d info %d %d %d", h.status, h.info[0], h.info[1], h.info[2]);
        CUDA_TRY(cudaMemsetAsync(ws, 0, 16, stream));
        CUDA_TRY(cudaStreamSynchronize(stream));
        if (h.status == CARNATOR_ERR_DEVICE_TIMEOUT || h.status == CARNATOR_ERR_DEVICE_CHECK) return carnator_status(h.status);
        return CARNATOR_ERR_DEVICE_CHECK;
    }
    return CARNATOR_OK;
}

extern "C" carnator_status carnator_selftest_wait_timeout(void* ws, uint64_t limit_ns, void* stream_) {
    if (!ws || !aligned(ws, 256)) return CARNATOR_ERR_WORKSPACE;
    if (limit_ns == 0 || limit_ns > kDefaultWaitNs) return CARNATOR_ERR_INVALID_ARG;
    carnator_status st = check_device();
    if (st != CARNATOR_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(WsHeader), stream));
    tc::wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(static_cast<WsHeader*>(ws), limit_ns);
    LAUNCH_CHECK("wait_timeout_selftest_kernel");
    return CARNATOR_OK;
}

extern "C" const char* carnator_status_string(carnator_status s) {
    switch (s) {
        case CARNATOR_OK: return "ok";
        case CARNATOR_ERR_INVALID_ARG: return "invalid argument";
        case CARNATOR_ERR_UNSUPPORTED: return "unsupported shape or device";
        case CARNATOR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CARNATOR_ERR_CUDA: return "CUDA call failed";
        case CARNATOR_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
        case CARNATOR_ERR_DEVICE_CHECK: return "device-side consistency check failed";
    }
    return "unknown status";
}

extern "C" const char* carnator_last_cuda_error(void) { return g_cuda_error; }
extern "C" int64_t carnator_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }
extern "C" int32_t carnator_version(void) { return 1; }
