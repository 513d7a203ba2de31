// Connectivity builder kernels: block pooling (HBM-bound), pooled-score tile product (fp32 FFMA),
// per-row selection (top-k or cumulative softmax mass) with the always-kept blocks.
// Paper: Appendix "Reuse-Scope Implementation Details" (per head and query block, the smallest set of
// key blocks covering a fixed fraction of the attention mass), in the pooled-score form.
#pragma once
#include "common.cuh"

namespace carnator {

// ----------------------------------------------------------------------------------------------
// M1: block means of Q and K.  One CTA per (tensor, b, h, block); reads block x D bf16 once.
// ----------------------------------------------------------------------------------------------
struct PoolArgs {
    const __nv_bfloat16* X[2];
    int64_t stride[2][3];
    int block[2];
    int nb[2];
    float* out[2];     // [B,H,nb,D]
    int N, H;
};

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <int D>
__global__ void __launch_bounds__(256) pool_kernel(PoolArgs a) {
    constexpr int TPR = D / 8;          // threads per token row (16 B each)
    constexpr int RPP = 256 / TPR;      // token rows per pass
    const int which = blockIdx.z & 1;
    const int b = blockIdx.z >> 1;
    const int h = blockIdx.y;
    const int I = blockIdx.x;
    // select with ternaries: dynamic indexing of the argument struct would force a local copy
    const int nb = which ? a.nb[1] : a.nb[0];
    if (I >= nb) return;
    const int block = which ? a.block[1] : a.block[0];
    const __nv_bfloat16* X = which ? a.X[1] : a.X[0];
    float* out = which ? a.out[1] : a.out[0];
    const int64_t sb = which ? a.stride[1][0] : a.stride[0][0];
    const int64_t sh = which ? a.stride[1][1] : a.stride[0][1];
    const int64_t sn = which ? a.stride[1][2] : a.stride[0][2];
    const int tok0 = I * block;
    const int nvalid = min(block, a.N - tok0);
    const int r = threadIdx.x / TPR, c = threadIdx.x % TPR;
    const __nv_bfloat16* base = X + b * sb + h * sh + int64_t(tok0) * sn + c * 8;

    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    // rows r, r+RPP, ...; issue up to four independent 16-byte loads before using them
    for (int row0 = r; row0 < nvalid; row0 += 4 * RPP) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            int row = row0 + u * RPP;
            v[u] = (row < nvalid) ? ld_stream16(base + int64_t(row) * sn) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc[2 * e]     += __uint_as_float(w[e] << 16);
                acc[2 * e + 1] += __uint_as_float(w[e] & 0xFFFF0000u);
            }
        }
    }

    __shared__ float red[RPP][D + 4];
#pragma unroll
    for (int e = 0; e < 8; ++e) red[r][c * 8 + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll
        for (int rr = 0; rr < RPP; ++rr) s += red[rr][threadIdx.x];
        out[((int64_t(b) * a.H + h) * nb + I) * D + threadIdx.x] = s / float(nvalid);
    }
}

// ----------------------------------------------------------------------------------------------
// M2: S[I,J] = scale * <qbar_I, kbar_J>, plain fp32 FFMA (no tensor-core rounding), 64x64 tile per CTA.
// ----------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) score_kernel(const float* __restrict__ qbar, const float* __restrict__ kbar,
                                                    float* __restrict__ scores, int nqb, int nkb, float scale) {
    constexpr int TM = 64, TN = 64, TK = 16;
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int bh = blockIdx.z;
    const int i0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
    const float* A = qbar + int64_t(bh) * nqb * D;
    const float* Bm = kbar + int64_t(bh) * nkb * D;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    // loader mapping: 256 threads move a 64 x 16 slab (float4 per thread)
    const int lrow = threadIdx.x / 4, lcol = (threadIdx.x % 4) * 4;
    for (int k0 = 0; k0 < D; k0 += TK) {
        float4 va = make_float4(0, 0, 0, 0), vb = make_float4(0, 0, 0, 0);
        if (i0 + lrow < nqb) va = *reinterpret_cast<const float4*>(A + int64_t(i0 + lrow) * D + k0 + lcol);
        if (j0 + lrow < nkb) vb = *reinterpret_cast<const float4*>(Bm + int64_t(j0 + lrow) * D + k0 + lcol);
        As[lcol + 0][lrow] = va.x; As[lcol + 1][lrow] = va.y; As[lcol + 2][lrow] = va.z; As[lcol + 3][lrow] = va.w;
        Bs[lcol + 0][lrow] = vb.x; Bs[lcol + 1][lrow] = vb.y; Bs[lcol + 2][lrow] = vb.z; Bs[lcol + 3][lrow] = vb.w;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[k][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Bs[k][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int I = i0 + ty * 4 + i;
        if (I >= nqb) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int J = j0 + tx * 4 + j;
            if (J < nkb) scores[(int64_t(bh) * nqb + I) * nkb + J] = scale * acc[i][j];
        }
    }
}

// ----------------------------------------------------------------------------------------------
// M3: per-row selection.
// ----------------------------------------------------------------------------------------------
__device__ __forceinline__ bool forced_block(int I, int J, const Geometry& g) {
    if (g.text_dense && g.n_text > 0 && (I * g.bq < g.n_text || J * g.bk < g.n_text)) return true;
    if (g.window >= 0) {
        int q_lo = max(I * g.bq, g.n_text), q_hi = min(g.N, (I + 1) * g.bq) - 1;
        int k_lo = max(J * g.bk, g.n_text), k_hi = min(g.N, (J + 1) * g.bk) - 1;
        if (q_hi >= q_lo && k_hi >= k_lo) {
            int f_lo = max(0, (q_lo - g.n_text) / g.hw - g.window);
            int f_hi = min(g.T - 1, (q_hi - g.n_text) / g.hw + g.window);
            int kf_lo = (k_lo - g.n_text) / g.hw, kf_hi = (k_hi - g.n_text) / g.hw;
            if (kf_lo <= f_hi && kf_hi >= f_lo) return true;
        }
    }
    return false;
}

__device__ __forceinline__ uint32_t ordered_bits(float s) {
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ int topk_count_dev(float ratio, int n) {
    if (n <= 0) return 0;
    double x = __dsub_rn(__dmul_rn(double(ratio), double(n)), 1e-6);
    int k = int(ceil(x));
    return max(1, min(n, k));
}

template <typename T>
__device__ __forceinline__ T block_sum(T v, T* scratch /* >= 8 */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    T t = 0;
    for (int w = 0; w < int(blockDim.x >> 5); ++w) t += scratch[w];
    return t;
}

struct SelectArgs {
    const float* scores;   // [B,H,nqb,nkb]
    uint8_t* mask;         // [B,H,nqb,nkb]
    int nqb, nkb, npad, H;
    int mode;
    float keep_ratio, mass;
    int count_includes_forced;
    int k_all;             // top-k count over all nkb blocks (host computed)
    int values_are_mass;   // cumulative-mass mode on non-negative block masses: p = value / sum instead of a softmax
    Geometry g;
};

// One CTA (256 threads) per (b,h,I).  Dynamic shared memory: npad uint64 sort keys + nkb keep bytes
// (+ npad doubles for the cumulative-mass mode).
__global__ void __launch_bounds__(256) select_kernel(SelectArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
    double* pm = reinterpret_cast<double*>(smem_raw + size_t(a.npad) * 8);                 // only in cumulative-mass mode
    uint8_t* keep = smem_raw + size_t(a.npad) * 8 * (a.mode == CARNATOR_MODE_CUMMASS ? 2 : 1);
    __shared__ double dscratch[8];
    __shared__ int iscratch[8];
    __shared__ float fscratch[8];

    const int I = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int64_t row = ((int64_t(b) * a.H + h) * a.nqb + I) * a.nkb;
    const float* s = a.scores + row;
    const int tid = threadIdx.x, nt = blockDim.x;

    // keys: score-ordered bits, ties -> lower J first.  Always-kept and padding entries get key 0 (sort last).
    int my_forced = 0;
    float my_max = -INFINITY;
    for (int J = tid; J < a.npad; J += nt) {
        unsigned long long key = 0ull;
        if (J < a.nkb) {
            bool f = forced_block(I, J, a.g);
            float v = s[J];
            my_max = fmaxf(my_max, v);
            keep[J] = f ? 1 : 0;
            my_forced += f ? 1 : 0;
            if (!f) key = (static_cast<unsigned long long>(ordered_bits(v)) << 32) | (0xFFFFFFFFu - uint32_t(J));
        }
        keys[J] = key;
    }
    const int nforced = block_sum<int>(my_forced, iscratch);
    const int nfree = a.nkb - nforced;

    // bitonic sort, descending
    for (int k = 2; k <= a.npad; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            __syncthreads();
            for (int i = tid; i < a.npad; i += nt) {
                int ixj = i ^ j;
                if (ixj > i) {
                    unsigned long long x = keys[i], y = keys[ixj];
                    bool desc = ((i & k) == 0);
                    if (desc ? (x < y) : (x > y)) { keys[i] = y; keys[ixj] = x; }
                }
            }
        }
    }
    __syncthreads();

    int n_admit = 0;
    if (a.mode == CARNATOR_MODE_TOPK) {
        n_admit = a.count_includes_forced ? max(0, a.k_all - nforced) : topk_count_dev(a.keep_ratio, nfree);
        n_admit = min(n_admit, nfree);
    } else {
        // row max (block reduce), softmax mass in fp64
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) my_max = fmaxf(my_max, __shfl_xor_sync(0xffffffffu, my_max, o));
        if ((tid & 31) == 0) fscratch[tid >> 5] = my_max;
        __syncthreads();
        float rmax = fscratch[0];
        for (int w = 1; w < (nt >> 5); ++w) rmax = fmaxf(rmax, fscratch[w]);
        double my_all = 0.0, my_fm = 0.0;
        for (int J = tid; J < a.nkb; J += nt) {
            double e = a.values_are_mass ? double(s[J]) : exp(double(s[J]) - double(rmax));
            my_all += e;
            if (keep[J]) my_fm += e;
        }
        const double total = block_sum<double>(my_all, dscratch);
        const double forced_mass = block_sum<double>(my_fm, dscratch) / total;
        // p of the sorted free blocks, then an exclusive prefix sum in sorted order
        const int per = a.npad / nt > 0 ? a.npad / nt : 1;
        for (int t = tid; t < a.npad; t += nt) {
            double p = 0.0;
            if (t < nfree) {
                int J = int(0xFFFFFFFFu - uint32_t(keys[t] & 0xFFFFFFFFull));
                p = (a.values_are_mass ? double(s[J]) : exp(double(s[J]) - double(rmax))) / total;
            }
            pm[t] = p;
        }
        __syncthreads();
        // chunked scan: thread t owns [t*per, (t+1)*per)
        double chunk = 0.0;
        const int c0 = tid * per;
        if (c0 < a.npad) for (int t = c0; t < c0 + per && t < a.npad; ++t) chunk += pm[t];
        __shared__ double chunk_sums[256];
        chunk_sums[tid] = chunk;
        __syncthreads();
        double before = forced_mass;
        for (int t = 0; t < tid; ++t) before += chunk_sums[t];
        // admitted iff the mass kept before this block is still below the target
        int my_admit = 0;
        const double target = double(a.mass);
        if (c0 < a.npad) {
            double run = before;
            for (int t = c0; t < c0 + per && t < a.npad; ++t) {
                if (t < nfree && run < target) my_admit++;
                run += pm[t];
            }
        }
        n_admit = block_sum<int>(my_admit, iscratch);
    }

    for (int t = tid; t < n_admit; t += nt) {
        int J = int(0xFFFFFFFFu - uint32_t(keys[t] & 0xFFFFFFFFull));
        keep[J] = 1;
    }
    __syncthreads();
    for (int J = tid; J < a.nkb; J += nt) a.mask[row + J] = keep[J];
}

// Top-k mode without a sort: one warp per (b,h,I).  Each lane keeps the order-preserving keys of the
// blocks J = lane, lane+32, ... in registers; the k-th largest key is found bit by bit (largest T with
// #(key >= T) >= k), then equal keys are admitted in ascending block order until k is reached.
template <int NPL>   // keys per lane: nkb <= 32 * NPL
__global__ void __launch_bounds__(256) select_topk_kernel(SelectArgs a, int rows) {
    // frame span of every key block, computed once per CTA (two integer divisions per block)
    extern __shared__ int2 kframes[];
    const Geometry g = a.g;
    for (int J = threadIdx.x; J < a.nkb; J += blockDim.x) {
        const int k_lo = max(J * g.bk, g.n_text), k_hi = min(g.N, (J + 1) * g.bk) - 1;
        kframes[J] = (k_hi >= k_lo) ? make_int2((k_lo - g.n_text) / g.hw, (k_hi - g.n_text) / g.hw) : make_int2(1, 0);
    }
    __syncthreads();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= rows) return;
    const int I = warp % a.nqb;
    const int64_t row = int64_t(warp) * a.nkb;
    const float* s = a.scores + row;

    // the query block's side of the always-kept rule
    const bool text_row = g.text_dense && g.n_text > 0 && I * g.bq < g.n_text;
    const int text_cols = (g.text_dense && g.n_text > 0) ? (g.n_text + g.bk - 1) / g.bk : 0;   // key blocks holding text
    int f_lo = 0, f_hi = 0;
    bool has_window = false;                   // the query block holds video tokens and a window is asked for
    if (g.window >= 0) {
        const int q_lo = max(I * g.bq, g.n_text), q_hi = min(g.N, (I + 1) * g.bq) - 1;
        if (q_hi >= q_lo) {
            has_window = true;
            f_lo = max(0, (q_lo - g.n_text) / g.hw - g.window);
            f_hi = min(g.T - 1, (q_hi - g.n_text) / g.hw + g.window);
        }
    }

    uint32_t key[NPL];
    uint32_t forced_bits[(NPL + 31) / 32];
#pragma unroll
    for (int w = 0; w < (NPL + 31) / 32; ++w) forced_bits[w] = 0u;
    int my_forced = 0;
#pragma unroll
    for (int t = 0; t < NPL; ++t) {
        const int J = t * 32 + lane;
        uint32_t k = 0u;                       // always-kept and out-of-range entries never compete
        if (J < a.nkb) {
            const int2 kf = kframes[J];
            const bool forced = text_row || J < text_cols || (has_window && kf.x <= kf.y && kf.x <= f_hi && kf.y >= f_lo);
            if (forced) { forced_bits[t >> 5] |= 1u << (t & 31); ++my_forced; }
            else k = ordered_bits(s[J]);
        }
        key[t] = k;
    }
    int nforced = my_forced;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nforced += __shfl_xor_sync(0xffffffffu, nforced, o);
    const int nfree = a.nkb - nforced;
    int n_admit = a.count_includes_forced ? max(0, a.k_all - nforced) : topk_count_dev(a.keep_ratio, nfree);
    n_admit = min(n_admit, nfree);

    uint32_t T = 0xFFFFFFFFu;                  // nothing admitted by score
    int need_eq = 0;
    if (n_admit > 0) {
        T = 0u;
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = T | (1u << bit);
            int c = 0;
#pragma unroll
            for (int t = 0; t < NPL; ++t) c += (key[t] >= cand) ? 1 : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            if (c >= n_admit) T = cand;
        }
        int gt = 0;
#pragma unroll
        for (int t = 0; t < NPL; ++t) gt += (key[t] > T) ? 1 : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gt += __shfl_xor_sync(0xffffffffu, gt, o);
        need_eq = n_admit - gt;                // >= 1 blocks with key == T, lowest block index first
    }
    int seen_eq = 0;
#pragma unroll
    for (int t = 0; t < NPL; ++t) {
        const int J = t * 32 + lane;
        const bool eq = (n_admit > 0) && key[t] == T;
        const unsigned bal = __ballot_sync(0xffffffffu, eq);
        const int rank = seen_eq + __popc(bal & ((1u << lane) - 1u));
        seen_eq += __popc(bal);
        const bool keep = ((forced_bits[t >> 5] >> (t & 31)) & 1u) || (n_admit > 0 && key[t] > T) || (eq && rank < need_eq);
        if (J < a.nkb) a.mask[row + J] = keep ? 1 : 0;
    }
}


}  // namespace carnator
