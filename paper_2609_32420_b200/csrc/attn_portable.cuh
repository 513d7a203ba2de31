// Portable block-sparse attention kernel (mma.sync m16n8k16, cp.async double buffering).
// Handles every supported shape (D in {64,128}, blocks in {64,128}); it is the bring-up path and the
// executor for shapes the tcgen05 kernel does not take.  Steps S1-S3: S = scale*Q K^T on the listed
// key blocks, online softmax, O += P V, O /= l, LSE = m + ln l.
// Paper: Section 3.3, "Historical Sparse-Connectivity Reuse".
#pragma once
#include "common.cuh"

namespace carnator {

struct AttnArgs {
    const __nv_bfloat16 *Q, *K, *V;
    __nv_bfloat16* O;
    float* LSE;                       // [B,H,N]
    int64_t qs[3], ks[3], vs[3], os[3];
    const int32_t *counts, *order, *lists;
    WsHeader* hdr;
    int B, H, N, nqb, nkb, block_q, block_k;
    float scale_log2;                 // softmax_scale * log2(e)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;   // size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D, int BQ>
struct PortableCfg {
    static constexpr int KC = 64;                 // keys per chunk
    static constexpr int LD = D + 8;              // padded row (elements): ldmatrix rows fall in distinct banks
    static constexpr int NW = BQ / 16;            // warps; each owns 16 query rows
    static constexpr int NT = NW * 32;
    static constexpr size_t smem_bytes = size_t(BQ + 4 * KC) * LD * 2;
};

template <int D, int BQ>
__global__ void __launch_bounds__(BQ * 2) attn_portable_kernel(AttnArgs a) {
    using C = PortableCfg<D, BQ>;
    constexpr int KC = C::KC, LD = C::LD, NT = C::NT;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* sK = sQ + BQ * LD;             // [2][KC][LD]
    __nv_bfloat16* sV = sK + 2 * KC * LD;         // [2][KC][LD]

    const int b = blockIdx.z, h = blockIdx.y;
    const int64_t bh = int64_t(b) * a.H + h;
    const int I = a.order[bh * a.nqb + blockIdx.x];
    const int count = a.counts[bh * a.nqb + I];
    if (count < 0) return;                         // skipped query block (region-restricted form): output untouched
    const int32_t* list = a.lists + (bh * a.nqb + I) * int64_t(a.nkb);
    const int q0 = I * BQ;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tig = lane & 3;
    {
        // The lists are only as good as the workspace they were read from: a count beyond nkb, an index outside
        // [0, nkb) or a list that does not ascend stops this query block before anything is loaded.
        int bad = count > a.nkb ? 1 : 0;
        for (int i = tid; i < min(count, a.nkb); i += NT) {
            const int J = list[i];
            if (J < 0 || J >= a.nkb || (i > 0 && J <= list[i - 1])) bad = 1;
        }
        if (__syncthreads_or(bad)) {
            if (tid == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_CHECK, 22, I, blockIdx.x);
            return;
        }
    }

    const __nv_bfloat16* Qp = a.Q + b * a.qs[0] + h * a.qs[1];
    const __nv_bfloat16* Kp = a.K + b * a.ks[0] + h * a.ks[1];
    const __nv_bfloat16* Vp = a.V + b * a.vs[0] + h * a.vs[1];

    const int cpb = a.block_k / KC;               // chunks per key block
    const int nchunks = count * cpb;

    auto load_kv = [&](int chunk, int stage) {
        const int J = list[chunk / cpb];
        const int key0 = J * a.block_k + (chunk % cpb) * KC;
        constexpr int VEC = D / 8;
        for (int idx = tid; idx < KC * VEC; idx += NT) {
            const int r = idx / VEC, c = idx % VEC;
            const int key = key0 + r;
            const bool ok = key < a.N;
            const int64_t kk = ok ? key : 0;
            cp_async16(smem_u32(sK + (stage * KC + r) * LD + c * 8), Kp + kk * a.ks[2] + c * 8, ok);
            cp_async16(smem_u32(sV + (stage * KC + r) * LD + c * 8), Vp + kk * a.vs[2] + c * 8, ok);
        }
    };

    // Q tile (rows >= N are zero) together with the first K/V chunk
    {
        constexpr int VEC = D / 8;
        for (int idx = tid; idx < BQ * VEC; idx += NT) {
            const int r = idx / VEC, c = idx % VEC;
            const bool ok = q0 + r < a.N;
            const int64_t qq = ok ? q0 + r : 0;
            cp_async16(smem_u32(sQ + r * LD + c * 8), Qp + qq * a.qs[2] + c * 8, ok);
        }
    }
    if (nchunks > 0) load_kv(0, 0);
    cp_async_commit();

    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    uint32_t qf[D / 16][4];

    for (int chunk = 0; chunk < nchunks; ++chunk) {
        const int stage = chunk & 1;
        if (chunk + 1 < nchunks) load_kv(chunk + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        if (chunk == 0) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
                ldmatrix_x4(qf[kk], smem_u32(sQ + (warp * 16 + (lane & 15)) * LD + kk * 16 + (lane >> 4) * 8));
        }

        const int J = list[chunk / cpb];
        const int key0 = J * a.block_k + (chunk % cpb) * KC;
        if (key0 < a.N) {
            const __nv_bfloat16* cK = sK + stage * KC * LD;
            const __nv_bfloat16* cV = sV + stage * KC * LD;
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
            // scale into the log2 domain, exclude keys >= N
            const bool tail = key0 + KC > a.N;
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int i = 0; i < KC / 8; ++i) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = s[i][e] * a.scale_log2;
                    if (tail && key0 + i * 8 + 2 * tig + (e & 1) >= a.N) v = -INFINITY;
                    s[i][e] = v;
                    mx[e >> 1] = fmaxf(mx[e >> 1], v);
                }
            }
            float alpha[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                const float m_new = fmaxf(m_run[r], mx[r]);      // finite: the chunk holds a valid key
                alpha[r] = exp2f(m_run[r] - m_new);               // first chunk: exp2(-inf) = 0
                m_run[r] = m_new;
                l_run[r] *= alpha[r];
            }
#pragma unroll
            for (int i = 0; i < KC / 8; ++i) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float p = exp2f(s[i][e] - m_run[e >> 1]);
                    s[i][e] = p;
                    l_run[e >> 1] += p;
                }
            }
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
                o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
            }
#pragma unroll
            for (int ks = 0; ks < KC / 16; ++ks) {
                uint32_t pa[4];
                pa[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
                pa[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
                pa[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
                pa[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
                for (int dp = 0; dp < D / 16; ++dp) {
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, smem_u32(cV + (ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + dp * 16 + (lane >> 4) * 8));
                    mma_bf16(o[2 * dp], pa, vb[0], vb[1]);
                    mma_bf16(o[2 * dp + 1], pa, vb[2], vb[3]);
                }
            }
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }
    cp_async_wait<0>();

    // epilogue
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = q0 + warp * 16 + g + r * 8;
        if (row >= a.N) continue;
        const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
        __nv_bfloat16* op = a.O + b * a.os[0] + h * a.os[1] + int64_t(row) * a.os[2];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            const uint32_t v = pack_bf16(o[i][2 * r] * inv, o[i][2 * r + 1] * inv);
            *reinterpret_cast<uint32_t*>(op + i * 8 + 2 * tig) = v;
        }
        if (tig == 0)
            a.LSE[bh * a.N + row] = l_run[r] > 0.f ? (m_run[r] + log2f(l_run[r])) * kLn2 : -INFINITY;
    }
}

}  // namespace carnator
