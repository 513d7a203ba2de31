// Seeded self-attention expansion of the Early-Signature localisation:
//   S_i = mean_h [ max_{u in I+} A_h[i,u] - max_{u in I-} A_h[i,u] ],   A_h[i,u] = exp(s_iu - LSE_i),
// with I+ / I- the noun and background seed token sets (Section 3.2, evidence region construction;
// Appendix "Evidence Region Construction").  exp is monotone, so per head only the largest score over each
// seed set is needed: a Q x K_seed^T product on gathered key rows followed by row maxima, then one exponential
// per query, head and set.  This file holds the mma.sync form, which streams the seed rows in chunks of 64 and takes
// any number of them; calls with at most 512 seeds run on the tcgen05 kernel of seed_expand_tcgen05.cuh instead.
#pragma once
#include "attn_portable.cuh"

namespace carnator {

struct SeedArgs {
    const __nv_bfloat16 *Q, *K;
    int64_t qs[3], ks[3];
    const float* LSE;        // [B,H,N], natural log, of the dense self-attention
    const int32_t* seeds;    // [n_pos + n_neg] token indices, positives first
    int n_pos, n_neg;
    float* per_head;         // [B,H,N]
    int B, H, N;
    float scale_log2;
};

template <int D>
__global__ void __launch_bounds__(256) seed_expand_kernel(SeedArgs a) {
    constexpr int BQ = 128, KC = 64, LD = D + 8, NT = 256;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* sK = sQ + BQ * LD;             // [2][KC][LD]
    const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * BQ;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tig = lane & 3;
    const __nv_bfloat16* Qp = a.Q + b * a.qs[0] + h * a.qs[1];
    const __nv_bfloat16* Kp = a.K + b * a.ks[0] + h * a.ks[1];
    const int cpos = (a.n_pos + KC - 1) / KC, cneg = (a.n_neg + KC - 1) / KC;
    const int nchunks = cpos + cneg;

    // chunk c covers entries [e0, e0 + 64) of the positive list (c < cpos) or of the negative list
    auto chunk_range = [&](int c, int& base, int& len) {
        if (c < cpos) { base = c * KC; len = min(KC, a.n_pos - c * KC); }
        else { base = a.n_pos + (c - cpos) * KC; len = min(KC, a.n_neg - (c - cpos) * KC); }
    };
    auto load_k = [&](int c, int stage) {
        int base, len;
        chunk_range(c, base, len);
        constexpr int VEC = D / 8;
        for (int idx = tid; idx < KC * VEC; idx += NT) {
            const int r = idx / VEC, v = idx % VEC;
            int tok = (r < len) ? a.seeds[base + r] : -1;
            const bool ok = tok >= 0 && tok < a.N;
            cp_async16(smem_u32(sK + (stage * KC + r) * LD + v * 8), Kp + int64_t(ok ? tok : 0) * a.ks[2] + v * 8, ok);
        }
    };
    {
        constexpr int VEC = D / 8;
        for (int idx = tid; idx < BQ * VEC; idx += NT) {
            const int r = idx / VEC, v = idx % VEC;
            const bool ok = q0 + r < a.N;
            cp_async16(smem_u32(sQ + r * LD + v * 8), Qp + int64_t(ok ? q0 + r : 0) * a.qs[2] + v * 8, ok);
        }
    }
    if (nchunks > 0) load_k(0, 0);
    cp_async_commit();

    float mpos[2] = {-INFINITY, -INFINITY}, mneg[2] = {-INFINITY, -INFINITY};
    uint32_t qf[D / 16][4];
    for (int c = 0; c < nchunks; ++c) {
        const int stage = c & 1;
        if (c + 1 < nchunks) load_k(c + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        if (c == 0) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
                ldmatrix_x4(qf[kk], smem_u32(sQ + (warp * 16 + (lane & 15)) * LD + kk * 16 + (lane >> 4) * 8));
        }
        const __nv_bfloat16* cK = sK + stage * KC * LD;
        float s[KC / 8][4];
#pragma unroll
        for (int i = 0; i < KC / 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
            for (int np = 0; np < KC / 16; ++np) {
                uint32_t kb[4];
                ldmatrix_x4(kb, smem_u32(cK + (np * 16 + (lane & 7) + ((lane >> 4) << 3)) * LD + kk * 16 + ((lane >> 3) & 1) * 8));
                mma_bf16(s[2 * np], qf[kk], kb[0], kb[1]);
                mma_bf16(s[2 * np + 1], qf[kk], kb[2], kb[3]);
            }
        }
        int base, len;
        chunk_range(c, base, len);
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < KC / 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (i * 8 + 2 * tig + (e & 1) < len) mx[e >> 1] = fmaxf(mx[e >> 1], s[i][e]);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (c < cpos) mpos[r] = fmaxf(mpos[r], mx[r]); else mneg[r] = fmaxf(mneg[r], mx[r]);
        }
        __syncthreads();
    }
    cp_async_wait<0>();
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        mpos[r] = fmaxf(mpos[r], __shfl_xor_sync(0xffffffffu, mpos[r], 1));
        mpos[r] = fmaxf(mpos[r], __shfl_xor_sync(0xffffffffu, mpos[r], 2));
        mneg[r] = fmaxf(mneg[r], __shfl_xor_sync(0xffffffffu, mneg[r], 1));
        mneg[r] = fmaxf(mneg[r], __shfl_xor_sync(0xffffffffu, mneg[r], 2));
        const int row = q0 + warp * 16 + g + r * 8;
        if (tig == 0 && row < a.N) {
            const int64_t o = (int64_t(b) * a.H + h) * a.N + row;
            const float l2 = a.LSE[o] * kLog2e;
            // an empty seed set contributes 0 (max over nothing)
            const float pp = a.n_pos > 0 ? exp2f(mpos[r] * a.scale_log2 - l2) : 0.f;
            const float pn = a.n_neg > 0 ? exp2f(mneg[r] * a.scale_log2 - l2) : 0.f;
            a.per_head[o] = pp - pn;
        }
    }
}

// mean over heads, in head order (deterministic)
__global__ void __launch_bounds__(256) head_mean_kernel(const float* __restrict__ per_head, int B, int H, int N,
                                                        float* __restrict__ out) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= int64_t(B) * N) return;
    const int b = int(i / N), n = int(i % N);
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += per_head[(int64_t(b) * H + h) * N + n];
    out[i] = s / float(H);
}

}  // namespace carnator
