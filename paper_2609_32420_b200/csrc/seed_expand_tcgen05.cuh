// Seeded self-attention expansion on the tcgen05 tensor cores (Section 3.2, evidence region construction;
// Appendix "Evidence Region Construction"):
//   S_i = mean_h [ max_{u in I+} A_h[i,u] - max_{u in I-} A_h[i,u] ],   A_h[i,u] = exp(s_iu - LSE_i).
// exp is monotone, so a head needs, per query, only the largest raw score over each seed set and two exponentials.
//
// A first small kernel gathers the seed tokens' key rows of every head into one contiguous array (positives first,
// 512 rows per head, unused rows zero).  The main kernel is persistent: a CTA takes a contiguous range of (head,
// query tile) pairs, keeps the head's seed rows in shared memory (TMA, reloaded when the head changes), streams the
// query tiles through a two-slot ring (TMA) and multiplies each by the seed rows in chunks of 256 seeds
// (tcgen05.mma, M = 128 queries, N = 256 seeds: with N = 256 the query tile is read from shared memory half as often
// per flop as with N = 128, which keeps the products off the shared-memory bandwidth limit).  The scores of a chunk
// sit in tensor memory (two chunks of 256 fp32 columns = all 512 columns); two epilogue warpgroups take the tiles in
// turn, read the scores with tcgen05.ld and reduce them to the two maxima of their row.
// Every wait is bounded, as in the attention kernel.
#pragma once
#include "attn_tcgen05.cuh"

namespace carnator {
namespace tc {

constexpr int kSeedCap = 512;            // seeds per call that this kernel takes (two chunks of tensor memory)
constexpr int kSeedChunk = 256;          // seeds per product (N of the MMA) and per tensor-memory buffer
constexpr int kSeedThreads = 320;        // warps 0-7: two epilogue groups; warp 8: TMA producer; warp 9: MMA issuer

struct SeedTcArgs {
    const float* LSE;        // [B,H,N], natural log, of the dense self-attention
    float* per_head;         // [B,H,N]
    WsHeader* hdr;
    int n_pos, n_seeds;      // positives come first in the gathered rows
    int B, H, N, nqb;
    int tiles;               // B * H * nqb
    float scale_log2;
};

struct SeedGatherArgs {
    const __nv_bfloat16* K;
    int64_t ks[3];
    const int32_t* seeds;
    __nv_bfloat16* out;      // [B*H][kSeedCap][D]
    int n_seeds, H, N;
};

// one 16-byte piece per thread; rows past the seed count and seeds outside [0, N) become zero rows
template <int D>
__global__ void __launch_bounds__(256) seed_gather_kernel(SeedGatherArgs a) {
    constexpr int VEC = D / 8;
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx >= kSeedCap * VEC) return;
    const int r = idx / VEC, v = idx % VEC;
    const int h = blockIdx.y, b = blockIdx.z;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (r < a.n_seeds) {
        const int tok = a.seeds[r];
        if (tok >= 0 && tok < a.N)
            val = *reinterpret_cast<const uint4*>(a.K + b * a.ks[0] + h * a.ks[1] + int64_t(tok) * a.ks[2] + v * 8);
    }
    *reinterpret_cast<uint4*>(a.out + ((int64_t(b) * a.H + h) * kSeedCap + r) * D + v * 8) = val;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], both descriptors given as (low word, shared high word); converged warp, one elected
// lane issues (see mma_ts_el)
__device__ __forceinline__ void mma_ss_el(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "elect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}

template <int D>
struct SeedCfg {
    static constexpr int kBoxes = D / 64;
    static constexpr uint32_t kQBox = 128 * 128;                    // 128 query rows x 128 B
    static constexpr uint32_t kQTile = kBoxes * kQBox;
    static constexpr uint32_t kSBox = kSeedChunk * 128;             // 256 seed rows x 128 B
    static constexpr uint32_t kSTile = kBoxes * kSBox;              // one chunk of seeds
    static constexpr uint32_t kOffSeed = 0;
    static constexpr uint32_t kOffQ = (kSeedCap / kSeedChunk) * kSTile;
    static constexpr uint32_t kOffBar = kOffQ + 2 * kQTile;
    static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;    // barriers + slack to align the base to 1 KiB
};

template <int D>
__global__ void __launch_bounds__(kSeedThreads, 1)
seed_expand_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapSeed, const SeedTcArgs a) {
    using C = SeedCfg<D>;
    extern __shared__ unsigned char seed_smem[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(seed_smem) + 1023u) & ~1023u;
    const uint32_t sSeed = smem_base + C::kOffSeed, sQ = smem_base + C::kOffQ, bars = smem_base + C::kOffBar;
    auto bar_qfull = [&](int s) { return bars + 8 * s; };              // query tile in ring slot s has landed
    auto bar_qfree = [&](int s) { return bars + 16 + 8 * s; };         // every product of the tile in slot s has completed
    const uint32_t bar_seed = bars + 32, bar_drain = bars + 40;        // the head's seed rows have landed
    auto bar_sfull = [&](int g, int c) { return bars + 64 + 8 * (g * 2 + c); };   // chunk c of a tile of group g is in tensor memory
    auto bar_sfree = [&](int c) { return bars + 96 + 8 * c; };         // the tile's group has read chunk c
    volatile int* abortp = &abort_flag;
    const unsigned long long limit = a.hdr->wait_limit_ns ? a.hdr->wait_limit_ns : kDefaultWaitNs;

    // this CTA's tiles: a contiguous range of the (batch, head, query tile) order, so a head's seed rows are loaded
    // once per CTA that touches the head
    const int t_begin = int(int64_t(blockIdx.x) * a.tiles / gridDim.x);
    const int t_end = int(int64_t(blockIdx.x + 1) * a.tiles / gridDim.x);
    const int ntiles = t_end - t_begin;
    const int nchunks = (a.n_seeds + kSeedChunk - 1) / kSeedChunk;     // 1 or 2

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < 2; ++s) { mbar_init(bar_qfull(s), 1); mbar_init(bar_qfree(s), 1); mbar_init(bar_sfree(s), 4); }
        for (int g = 0; g < 2; ++g) for (int c = 0; c < 2; ++c) mbar_init(bar_sfull(g, c), 1);
        mbar_init(bar_seed, 1); mbar_init(bar_drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp == 8) {
        // ================= TMA producer: seed rows per head, query tiles =================
        if (lane == 0) {
            prefetch_tmap(&mapQ); prefetch_tmap(&mapSeed);
            int armed = -1;
            bool seed_armed = false;
            for (int n = 0; n < ntiles; ++n) {
                const int t = t_begin + n, s = n & 1;
                const int bh = t / a.nqb, I = t - bh * a.nqb;
                const int b = bh / a.H, h = bh - b * a.H;
                if (n == 0 || I == 0) {
                    // the seed rows of the previous head are in use until the products of its last tile have completed
                    if (n > 0 && !mbar_wait(bar_qfree((n - 1) & 1), uint32_t((n - 1) >> 1) & 1u, abortp, 64, limit)) {
                        set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 60, n, blockIdx.x); break;
                    }
                    mbar_expect_tx(bar_seed, uint32_t(nchunks) * C::kSTile);
                    for (int c = 0; c < nchunks; ++c)
#pragma unroll
                        for (int x = 0; x < C::kBoxes; ++x)
                            tma_load_2d(sSeed + c * C::kSTile + x * C::kSBox, &mapSeed, bar_seed, x * 64, bh * kSeedCap + c * kSeedChunk);
                    seed_armed = true;
                }
                if (n >= 2 && !mbar_wait(bar_qfree(s), uint32_t((n - 2) >> 1) & 1u, abortp, 64, limit)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 61, n, blockIdx.x); break;
                }
                mbar_expect_tx(bar_qfull(s), C::kQTile);              // rows >= N read as zero; their results are never stored
#pragma unroll
                for (int x = 0; x < C::kBoxes; ++x)
                    tma_load_4d(sQ + s * C::kQTile + x * C::kQBox, &mapQ, bar_qfull(s), x * 64, I * kBlock, h, b);
                armed = n;
            }
            if (*abortp) {      // copies in flight must land before the CTA gives its shared memory back
                for (int k = 0; k < 2 && armed - k >= 0; ++k)
                    mbar_wait_drain(bar_qfull((armed - k) & 1), uint32_t((armed - k) >> 1) & 1u, limit);
                if (seed_armed) mbar_wait_drain(bar_seed, 0, 20000000ull);     // either parity may be the pending one:
                if (seed_armed) mbar_wait_drain(bar_seed, 1, 20000000ull);     // one of the two returns at once
            }
        }
    } else if (warp == 9) {
        // ================= MMA issuer (converged warp, one elected lane issues) =================
        constexpr uint32_t idesc = instr_desc(kBlock, kSeedChunk, 0);
        const uint64_t dq = smem_desc(sQ, 16, 1024), ds = smem_desc(sSeed, 16, 1024);
        const uint32_t q_lo0 = uint32_t(dq), s_lo0 = uint32_t(ds), hi = uint32_t(dq >> 32);
        bool ok = true;
        int heads_seen = 0;
        for (int n = 0; n < ntiles && ok; ++n) {
            const int t = t_begin + n, s = n & 1, g = n & 1;
            const int I = t % a.nqb;
            if (n == 0 || I == 0) {
                ok = mbar_wait_warp(bar_seed, uint32_t(heads_seen) & 1u, abortp, 0, limit);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 62, n, blockIdx.x); break; }
                ++heads_seen;
            }
            ok = mbar_wait_warp(bar_qfull(s), uint32_t(n >> 1) & 1u, abortp, 0, limit);
            if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 63, n, blockIdx.x); break; }
            const uint32_t q_lo = q_lo0 + uint32_t(s) * (C::kQTile >> 4);
            for (int c = 0; c < nchunks && ok; ++c) {
                if (n >= 1) {       // the previous tile's group has read this chunk's scores out of tensor memory
                    ok = mbar_wait_warp(bar_sfree(c), uint32_t(n - 1) & 1u, abortp, 0, limit);
                    if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 64, n, blockIdx.x); break; }
                }
                tc_fence_after();
                const uint32_t s_lo = s_lo0 + uint32_t(c) * (C::kSTile >> 4), d_s = tmem + uint32_t(c * kSeedChunk);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t offq = ((kk / 4) * C::kQBox + (kk % 4) * 32) >> 4, offs = ((kk / 4) * C::kSBox + (kk % 4) * 32) >> 4;
                    mma_ss_el(d_s, q_lo + offq, s_lo + offs, hi, idesc, kk > 0 ? 1u : 0u);
                }
                tc_commit_el(bar_sfull(g, c));
            }
            if (ok) tc_commit_el(bar_qfree(s));
        }
        tc_commit_el(bar_drain);          // no product may still run when tensor memory is released
        mbar_wait_drain(bar_drain, 0, limit);
        __syncwarp();
    } else {
        // ================= epilogue: two warpgroups take the tiles in turn =================
        const int quarter = warp & 3, g = warp >> 2;
        const uint32_t lane_base = uint32_t(quarter * 32) << 16;
        bool ok = true;
        for (int n = g; n < ntiles && ok; n += 2) {
            const int t = t_begin + n;
            const int bh = t / a.nqb, I = t - bh * a.nqb;
            const int row = I * kBlock + quarter * 32 + lane;
            float mpos = -INFINITY, mneg = -INFINITY;
            for (int c = 0; c < nchunks && ok; ++c) {
                ok = mbar_wait_warp(bar_sfull(g, c), uint32_t(n >> 1) & 1u, abortp, 20, limit);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 65, n, blockIdx.x); break; }
                tc_fence_after();
#pragma unroll 1
                for (int grp = 0; grp < kSeedChunk / 32; ++grp) {
                    const int col0 = c * kSeedChunk + grp * 32;            // seed index of the group's first column
                    if (col0 >= a.n_seeds) break;                          // warp-uniform
                    float v[32];
                    tmem_ld32(tmem + lane_base + uint32_t(col0), v);
                    tmem_wait_ld();
                    if (col0 + 32 <= a.n_pos || (col0 >= a.n_pos && col0 + 32 <= a.n_seeds)) {
                        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // the whole group belongs to one set
#pragma unroll
                        for (int e = 0; e < 32; e += 2) m4[(e >> 1) & 3] = max3(m4[(e >> 1) & 3], v[e], v[e + 1]);
                        const float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                        if (col0 < a.n_pos) mpos = fmaxf(mpos, m); else mneg = fmaxf(mneg, m);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) {                      // the group straddles a set boundary or the end
                            const int u = col0 + e;
                            if (u < a.n_pos) mpos = fmaxf(mpos, v[e]);
                            else if (u < a.n_seeds) mneg = fmaxf(mneg, v[e]);
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive_warp(bar_sfree(c));
            }
            if (ok && row < a.N) {
                const int64_t o = int64_t(bh) * a.N + row;
                const float l2 = a.LSE[o] * kLog2e;
                // an empty seed set contributes 0 (max over nothing)
                const float pp = a.n_pos > 0 ? exp2f(mpos * a.scale_log2 - l2) : 0.f;
                const float pn = a.n_seeds > a.n_pos ? exp2f(mneg * a.scale_log2 - l2) : 0.f;
                a.per_head[o] = pp - pn;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

}  // namespace tc

// Shapes the tensor-core form takes; the others (more seeds, no seeds, a query tensor shared over heads or batch
// entries) run on the mma.sync kernel of seed_expand.cuh.
inline bool seed_tcgen05_supported(const carnator_shape* s, int n_seeds) {
    return (s->D == 64 || s->D == 128) && n_seeds > 0 && n_seeds <= tc::kSeedCap && tma_strides_ok(s, s->q_stride);
}

inline size_t seed_gather_bytes(const carnator_shape* s) { return size_t(s->B) * s->H * tc::kSeedCap * s->D * 2; }

template <int D>
inline carnator_status launch_seed_tc(const tc::SeedGatherArgs& ga, const tc::SeedTcArgs& a, const CUtensorMap& mq, const CUtensorMap& ms,
                                      int sms, cudaStream_t stream, char* err, size_t errlen) {
    using C = tc::SeedCfg<D>;
    dim3 ggrid((tc::kSeedCap * (D / 8) + 255) / 256, a.H, a.B);
    tc::seed_gather_kernel<D><<<ggrid, 256, 0, stream>>>(ga);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(err, errlen, "seed_gather_kernel: %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    auto kern = tc::seed_expand_tc_kernel<D>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(C::kSmemBytes));
    if (e != cudaSuccess) { snprintf(err, errlen, "cudaFuncSetAttribute(seed tcgen05): %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    const int grid = a.tiles < sms ? a.tiles : sms;
    kern<<<grid, tc::kSeedThreads, C::kSmemBytes, stream>>>(mq, ms, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(err, errlen, "seed_expand_tc_kernel: %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    return CARNATOR_OK;
}

}  // namespace carnator
