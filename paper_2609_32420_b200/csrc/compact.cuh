// C1: block mask (+ recompute rows) -> per-row ascending key-block lists, counts, and a per-head
// execution order (longest list first), so the attention kernel never fetches an empty tile.
// Paper: Appendix "Reuse-Scope Implementation Details" (connectivity is restricted before sparse
// execution) and "Latency Accounting" (in-loop mask / index lookups).
#pragma once
#include "common.cuh"

namespace carnator {

// One warp per (b,h,I).  grid.x = ceil(B*H*nqb / 8), 256 threads.
__global__ void __launch_bounds__(256) compact_rows_kernel(const uint8_t* __restrict__ mask,
                                                           const uint8_t* __restrict__ recompute,
                                                           int B, int H, int nqb, int nkb,
                                                           int32_t* __restrict__ counts,
                                                           int32_t* __restrict__ lists,
                                                           const uint8_t* __restrict__ active_q = nullptr,
                                                           const uint8_t* __restrict__ context_k = nullptr) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int rows = B * H * nqb;
    if (warp >= rows) return;
    const int I = warp % nqb;
    const int b = warp / (nqb * H);
    const bool dense = recompute != nullptr && recompute[b * nqb + I] != 0;
    // region-restricted form: a query block that is not active is skipped altogether (count -1: the attention
    // kernels leave its output rows untouched); listed key blocks must also be context blocks
    if (active_q != nullptr && active_q[b * nqb + I] == 0) {
        if (lane == 0) counts[warp] = -1;
        return;
    }
    const uint8_t* ctx = context_k != nullptr ? context_k + int64_t(b) * nkb : nullptr;
    const uint8_t* m = mask + int64_t(warp) * nkb;
    int32_t* out = lists + int64_t(warp) * nkb;
    int n = 0;
    for (int J0 = 0; J0 < nkb; J0 += 32) {
        int J = J0 + lane;
        bool on = (J < nkb) && (dense || m[J] != 0) && (ctx == nullptr || ctx[J] != 0);
        unsigned bal = __ballot_sync(0xffffffffu, on);
        if (on) out[n + __popc(bal & ((1u << lane) - 1u))] = J;
        n += __popc(bal);
    }
    if (lane == 0) counts[warp] = n;
}

// One CTA per (b,h): rank of row I = #{I' : c[I'] > c[I]} + #{I' < I : c[I'] == c[I]} (stable, deterministic).
__global__ void __launch_bounds__(256) order_rows_kernel(const int32_t* __restrict__ counts, int nqb,
                                                         int32_t* __restrict__ order, WsHeader* hdr) {
    extern __shared__ int32_t c[];
    const int bh = blockIdx.x;
    const int32_t* cnt = counts + int64_t(bh) * nqb;
    unsigned long long local = 0;
    for (int i = threadIdx.x; i < nqb; i += blockDim.x) { c[i] = cnt[i]; local += (unsigned long long)max(cnt[i], 0); }
    __syncthreads();
    for (int i = threadIdx.x; i < nqb; i += blockDim.x) {
        const int ci = c[i];
        int rank = 0;
        for (int j = 0; j < nqb; ++j) {
            int cj = c[j];
            rank += (cj > ci) || (cj == ci && j < i);
        }
        order[int64_t(bh) * nqb + rank] = i;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
    if ((threadIdx.x & 31) == 0 && local) atomicAdd(&hdr->tiles, local);
}

}  // namespace carnator
