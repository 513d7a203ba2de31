// Exact block attention mass on the tensor cores: for every (query block I, key block J) of a head,
//   mass[I,J] = (1/|I|) * sum_{i in I} sum_{j in J} exp(s_ij - LSE_i),
// the quantity the paper's connectivity rule is stated on (Appendix "Reuse-Scope Implementation Details":
// per head and query block, the smallest set of key blocks covering a fixed fraction of the attention
// mass).  LSE_i is the log-sum-exp of query i over all keys, as returned by a dense attention run.
//
// Same machinery as the attention kernel (TMA tiles with 128-byte swizzle, tcgen05.mma S = Q K^T into
// tensor memory, two softmax warpgroups taking the 128-key steps in turn), without V, P or O: four score
// buffers fill the 512 tensor-memory columns, so the MMA issuer runs well ahead of the exponentials.
// Every mbarrier wait is bounded (see attn_tcgen05.cuh).
#pragma once
#include "attn_tcgen05.cuh"

namespace carnator {
namespace tc {

constexpr int kMassSoftmaxWarps = 8;                        // two warpgroups taking the key blocks in turn
constexpr int kMassThreads = (kMassSoftmaxWarps + 4) * 32;  // third warpgroup: TMA producer, MMA issuer, two idle warps
constexpr int kMassWarpTma = 8, kMassWarpMma = 9;
constexpr int kMassTmemCols = 512;
constexpr int kMassSBufs = 4;      // score buffers (128 fp32 columns each)
constexpr int kMassStages = 4;     // K tile ring

struct MassArgs {
    const float* LSE;              // [B,H,N], natural log
    float* mass;                   // [B,H,nqb,nkb]
    WsHeader* hdr;
    int B, H, N, nqb, nkb;
    float scale_log2;
};

template <int D>
struct MassCfg {
    static constexpr int kBoxes = D / 64;
    static constexpr uint32_t kBoxBytes = kBlock * 128;
    static constexpr uint32_t kTileBytes = kBoxes * kBoxBytes;
    static constexpr uint32_t kOffQ = 0;
    static constexpr uint32_t kOffK = kTileBytes;
    static constexpr uint32_t kOffBar = kOffK + kMassStages * kTileBytes;
    static constexpr uint32_t kSmemBytes = kOffBar + 512 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kMassThreads, 1)
block_mass_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK, const MassArgs a) {
    using C = MassCfg<D>;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float red[2][8][4];          // [group][slot][lane quarter] partial sums of one (I,J) tile

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.z, h = blockIdx.y, I = blockIdx.x;
    const int64_t bh = int64_t(b) * a.H + h;
    const int T = a.nkb;                    // every key block is visited
    const int q0 = I * kBlock;
    const int nrows = min(kBlock, a.N - q0);

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + C::kOffQ;
    const uint32_t sK = smem_base + C::kOffK;
    const uint32_t bars = smem_base + C::kOffBar;
    const uint32_t bar_q = bars, bar_drain = bars + 8;
    auto bar_kfull = [&](int s) { return bars + 32 + 8 * s; };
    auto bar_kempty = [&](int s) { return bars + 64 + 8 * s; };
    auto bar_sfull = [&](int s) { return bars + 96 + 8 * s; };
    auto bar_sfree = [&](int s) { return bars + 128 + 8 * s; };
    auto bar_red = [&](int g, int s) { return bars + 160 + 8 * (g * 8 + s); };
    volatile int* abortp = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_q, 1); mbar_init(bar_drain, 1);
        for (int s = 0; s < kMassStages; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1); }
        for (int s = 0; s < kMassSBufs; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sfree(s), 4); }
        for (int g = 0; g < 2; ++g)
            for (int s = 0; s < 8; ++s) mbar_init(bar_red(g, s), 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMassWarpTma && lane == 0) { prefetch_tmap(&mapQ); prefetch_tmap(&mapK); }
    if (warp == kMassWarpMma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kMassTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp >= kMassSoftmaxWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
    if (warp == kMassWarpTma) {
        // ================= TMA producer: Q once, then every K tile of the head =================
        if (lane == 0) {
            mbar_expect_tx(bar_q, C::kTileBytes);
#pragma unroll
            for (int x = 0; x < C::kBoxes; ++x) tma_load_4d(sQ + x * C::kBoxBytes, &mapQ, bar_q, x * 64, q0, h, b);
            int armed = -1;
            for (int i = 0; i < T; ++i) {
                const int s = i % kMassStages;
                if (!mbar_wait(bar_kempty(s), (uint32_t(i / kMassStages) & 1u) ^ 1u, abortp, 32)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 31, i, blockIdx.x); break;
                }
                mbar_expect_tx(bar_kfull(s), C::kTileBytes);
#pragma unroll
                for (int x = 0; x < C::kBoxes; ++x)
                    tma_load_4d(sK + s * C::kTileBytes + x * C::kBoxBytes, &mapK, bar_kfull(s), x * 64, i * kBlock, h, b);
                armed = i;
            }
            if (*abortp) {      // copies in flight must land before the CTA gives its shared memory back
                mbar_wait_drain(bar_q, 0);
                for (int k = 0; k < kMassStages && armed - k >= 0; ++k)
                    mbar_wait_drain(bar_kfull((armed - k) % kMassStages), uint32_t((armed - k) / kMassStages) & 1u);
            }
        }
    } else if (warp == kMassWarpMma) {
        // ================= MMA issuer: S[i % 4] = Q K_i^T =================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kBlock, kBlock, 0);
            bool ok = mbar_wait(bar_q, 0, abortp);
            if (!ok) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 33, 0, blockIdx.x);
            for (int i = 0; i < T && ok; ++i) {
                const int s = i % kMassStages, sb = i % kMassSBufs;
                if (i >= kMassSBufs && !mbar_wait(bar_sfree(sb), uint32_t(i / kMassSBufs - 1) & 1u, abortp, 20)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 34, i, blockIdx.x); ok = false; break;
                }
                if (!mbar_wait(bar_kfull(s), uint32_t(i / kMassStages) & 1u, abortp, 20)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 35, i, blockIdx.x); ok = false; break;
                }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * C::kBoxBytes + (kk % 4) * 32;
                    mma_ss(tmem + sb * kBlock, smem_desc(sQ + off, 16, 1024),
                           smem_desc(sK + s * C::kTileBytes + off, 16, 1024), idesc_qk, kk > 0);
                }
                tc_commit(bar_sfull(sb));
                tc_commit(bar_kempty(s));
            }
            // tensor memory may only be released once every MMA has retired
            tc_commit(bar_drain);
            mbar_wait_drain(bar_drain, 0);
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
        // ================= exponentials and block sums (warps 0-7) =================
        const int quarter = warp & 3, wg = warp >> 2;
        const int r_loc = quarter * 32 + lane;
        const uint32_t lane_base = uint32_t(quarter * 32) << 16;
        const bool row_ok = r_loc < nrows;
        // exponent offset of this query: log2(e) * LSE_i; rows past N contribute nothing
        const float lse2 = row_ok ? a.LSE[bh * a.N + q0 + r_loc] * kLog2e : INFINITY;
        const float inv_rows = 1.f / float(nrows);
        bool ok = true;
        for (int i = wg; i < T; i += 2) {
            const int sb = i % kMassSBufs;
            ok = mbar_wait_warp(bar_sfull(sb), uint32_t(i / kMassSBufs) & 1u, abortp, 20);
            if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 36, i, blockIdx.x); break; }
            tc_fence_after();
            const int nvalid = min(kBlock, a.N - i * kBlock);
            const uint32_t tS = tmem + lane_base + sb * kBlock;
            float s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s[c]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive_warp(bar_sfree(sb));     // the scores are in registers: the buffer may be refilled
            // exp2(s * scale - lse2), two scores per FMA-pipe instruction; -inf offset for rows past N gives 0
            float v;
            if (nvalid == kBlock) {
                const uint64_t neg2 = pack2(-lse2, -lse2), scale2 = pack2(a.scale_log2, a.scale_log2);
                uint64_t part2[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float x0, x1;
                        unpack2(fma2(pack2(s[c][2 * e], s[c][2 * e + 1]), scale2, neg2), x0, x1);
                        part2[e & 3] = add2(part2[e & 3], pack2(ex2_approx(x0), ex2_approx(x1)));
                    }
                float p0, p1, p2, p3, p4, p5, p6, p7;
                unpack2(part2[0], p0, p1); unpack2(part2[1], p2, p3); unpack2(part2[2], p4, p5); unpack2(part2[3], p6, p7);
                v = ((p0 + p1) + (p2 + p3)) + ((p4 + p5) + (p6 + p7));
            } else {                              // the ragged last key block (warp-uniform): keys >= N never count
                const float neg = -lse2;
                float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float p = ex2_approx(fmaf(s[c][e], a.scale_log2, neg));
                        part[e & 3] += (c * 32 + e < nvalid) ? p : 0.f;
                    }
                v = (part[0] + part[1]) + (part[2] + part[3]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            // Four warps of the group -> one value; the first warp adds them in a fixed order.  It does so two of the
            // group's tiles later, when the other warps' arrivals are long past, so nobody stops for the hand-over
            // (eight slots per group: a warp can be two tiles ahead of the slowest warp of its group, no more, because
            // a score buffer is refilled only when all four have read it; a slot is rewritten eight tiles on).
            const int n = i >> 1;                       // this group's n-th tile
            if (lane == 0) red[wg][n & 7][quarter] = v;
            mbar_arrive_warp(bar_red(wg, n & 7));
            if (quarter == 0 && n >= 2) {
                const int m = n - 2;
                ok = mbar_wait_warp(bar_red(wg, m & 7), uint32_t(m >> 3) & 1u, abortp, 0);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 37, i, blockIdx.x); break; }
                if (lane == 0) {
                    const float tot = ((red[wg][m & 7][0] + red[wg][m & 7][1]) + red[wg][m & 7][2]) + red[wg][m & 7][3];
                    a.mass[(bh * a.nqb + I) * int64_t(a.nkb) + (2 * m + wg)] = tot * inv_rows;
                }
            }
        }
        // the group's last two tiles
        if (quarter == 0 && ok) {
            const int ntile = (T - wg + 1) / 2;         // tiles this group has handled
            for (int m = max(0, ntile - 2); m < ntile && ok; ++m) {
                ok = mbar_wait_warp(bar_red(wg, m & 7), uint32_t(m >> 3) & 1u, abortp, 0);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 37, m, blockIdx.x); break; }
                if (lane == 0) {
                    const float tot = ((red[wg][m & 7][0] + red[wg][m & 7][1]) + red[wg][m & 7][2]) + red[wg][m & 7][3];
                    a.mass[(bh * a.nqb + I) * int64_t(a.nkb) + (2 * m + wg)] = tot * inv_rows;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMassWarpMma) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kMassTmemCols) : "memory");
    }
}

}  // namespace tc

inline carnator_status launch_block_mass(const void* Q, const void* K, const int64_t qs[3], const int64_t ks[3],
                                         const tc::MassArgs& a, int D, cudaStream_t stream, char* err, size_t errlen) {
    CUtensorMap mq, mk;
    if (!tc::make_map(&mq, Q, a.B, a.H, a.N, D, qs, tc::kBlock) || !tc::make_map(&mk, K, a.B, a.H, a.N, D, ks, tc::kBlock)) {
        snprintf(err, errlen, "cuTensorMapEncodeTiled failed or is unavailable");
        return CARNATOR_ERR_CUDA;
    }
    dim3 grid(a.nqb, a.H, a.B);
    cudaError_t e;
    {   // the kernel's setmaxnreg split (40 / 232) needs 168 registers per thread at launch
        cudaFuncAttributes fa;
        e = (D == 128) ? cudaFuncGetAttributes(&fa, tc::block_mass_kernel<128>) : cudaFuncGetAttributes(&fa, tc::block_mass_kernel<64>);
        if (e != cudaSuccess) { snprintf(err, errlen, "cudaFuncGetAttributes(block_mass): %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
        if (fa.numRegs * tc::kMassThreads < tc::kMassSoftmaxWarps * 32 * 232 + 128 * 40) {
            snprintf(err, errlen, "block_mass_kernel was built with %d registers per thread: too few for its setmaxnreg split", fa.numRegs);
            return CARNATOR_ERR_UNSUPPORTED;
        }
    }
    if (D == 128) {
        e = cudaFuncSetAttribute(tc::block_mass_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(tc::MassCfg<128>::kSmemBytes));
        if (e == cudaSuccess) tc::block_mass_kernel<128><<<grid, tc::kMassThreads, tc::MassCfg<128>::kSmemBytes, stream>>>(mq, mk, a);
    } else {
        e = cudaFuncSetAttribute(tc::block_mass_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(tc::MassCfg<64>::kSmemBytes));
        if (e == cudaSuccess) tc::block_mass_kernel<64><<<grid, tc::kMassThreads, tc::MassCfg<64>::kSmemBytes, stream>>>(mq, mk, a);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(err, errlen, "block_mass_kernel: %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    return CARNATOR_OK;
}

}  // namespace carnator
