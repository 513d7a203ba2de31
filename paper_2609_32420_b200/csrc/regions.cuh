// Reuse-region kernels: evidence region -> active / context regions and blend weights, latent fusion,
// region -> block flags.  All memory-bound element-wise or small-stencil work.
// Paper: Section 3.3 "Region-Guided Latent Reuse" (Eq. latent reuse, weight W) and Appendix "Reuse-Scope
// Implementation Details" (dilation by 2 tokens, then by a further 3, per latent frame on the H x W grid;
// Chebyshev distance to the evidence region, normalised by the largest distance in the band, through smoothstep).
#pragma once
#include "common.cuh"

namespace carnator {

// One thread per token: Chebyshev distance to the nearest evidence token of the same frame, searched in the
// (2R+1)^2 window, R = r_active + r_context (255 = farther than R).  active = d <= r_active; context = d <= R
// (square neighbourhoods compose).  The largest distance inside the band goes to hdr->info[0] by atomicMax.
__global__ void __launch_bounds__(256) region_distance_kernel(const uint8_t* __restrict__ evidence, int T, int H, int W,
                                                              int r_active, int r_context, uint8_t* __restrict__ dist,
                                                              uint8_t* __restrict__ active, uint8_t* __restrict__ context,
                                                              WsHeader* hdr) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= T * H * W) return;
    const int x = n % W, y = (n / W) % H, t = n / (W * H);
    const int R = r_active + r_context;
    const uint8_t* f = evidence + int64_t(t) * H * W;
    int d = 255;
    for (int dy = -R; dy <= R; ++dy) {
        const int yy = y + dy;
        if (yy < 0 || yy >= H) continue;
        for (int dx = -R; dx <= R; ++dx) {
            const int xx = x + dx;
            if (xx < 0 || xx >= W) continue;
            if (f[yy * W + xx]) d = min(d, max(abs(dy), abs(dx)));
        }
    }
    dist[n] = uint8_t(d);
    active[n] = d <= r_active ? 1 : 0;
    context[n] = d <= R ? 1 : 0;
    if (d > 0 && d <= r_active) atomicMax(&hdr->info[0], d);
}

// W = 1 on the evidence region, 1 - smoothstep(d / d_max) on the band, 0 elsewhere.
__global__ void __launch_bounds__(256) region_weight_kernel(const uint8_t* __restrict__ dist, int n_tokens, int r_active,
                                                            const WsHeader* hdr, float* __restrict__ Wt) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= n_tokens) return;
    const int d = dist[n];
    float w = 0.f;
    if (d == 0) w = 1.f;
    else if (d <= r_active) {
        const float x = float(d) / float(hdr->info[0]);
        w = 1.f - (3.f * x * x - 2.f * x * x * x);
    }
    Wt[n] = w;
}

// z = W * z_target + (1 - W) * z_hist over [channels, tokens]; 16 bytes per thread and tensor.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) fuse_latents_kernel(const T* __restrict__ zt, const T* __restrict__ zh,
                                                           const float* __restrict__ Wt, int64_t channels, int64_t tokens,
                                                           T* __restrict__ out) {
    const int64_t nvec = tokens / VEC;                       // tokens % VEC == 0 is checked by the caller
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= channels * nvec) return;
    const int64_t c = i / nvec, v = i % nvec;
    const int64_t off = c * tokens + v * VEC;
    T a[VEC], b[VEC], o[VEC];
    *reinterpret_cast<uint4*>(a) = *reinterpret_cast<const uint4*>(zt + off);
    *reinterpret_cast<uint4*>(b) = *reinterpret_cast<const uint4*>(zh + off);
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const float w = Wt[v * VEC + e];
        const float r = w * float(a[e]) + (1.f - w) * float(b[e]);
        o[e] = T(r);
    }
    *reinterpret_cast<uint4*>(out + off) = *reinterpret_cast<const uint4*>(o);
}

// One warp per block of the token order (text tokens first): 1 if the block holds a token of the region.
__global__ void __launch_bounds__(256) region_block_flags_kernel(const uint8_t* __restrict__ region, int n_text, int n_video,
                                                                 int block, int text_value, int nblocks,
                                                                 uint8_t* __restrict__ flags) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= nblocks) return;
    const int t0 = warp * block, t1 = min(n_text + n_video, t0 + block);
    bool any = false;
    for (int t = t0 + lane; t < t1; t += 32) any |= (t < n_text) ? (text_value != 0) : (region[t - n_text] != 0);
    any = __any_sync(0xffffffffu, any);
    if (lane == 0) flags[warp] = any ? 1 : 0;
}

}  // namespace carnator
