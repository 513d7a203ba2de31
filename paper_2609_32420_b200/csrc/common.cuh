// Shared device/host helpers of the carnator library (workspace layout, status word, small math).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "carnator.h"

namespace carnator {

constexpr int kMaxKeyBlocksBuilder = 4096;   // select kernel sorts one row in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;   // limit of a bounded device-side wait unless the header says otherwise

// First 256 bytes of every workspace.
struct WsHeader {
    int32_t status;              // carnator_status set by kernels (0 = ok); first error wins
    int32_t info[3];             // where a bounded wait gave up / which check failed
    unsigned long long tiles;    // evaluated (query block, key block) pairs after compaction
    int32_t work[4];             // work-item counters of persistent kernels (zeroed with the header)
    unsigned long long wait_limit_ns;   // 0: the default limit of every bounded device-side wait; tests set a short one
    int32_t debug_withhold;      // 0 except in the test of the time-out path: the K producer withholds one copy
    int32_t pad[51];
};
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Layout of the attention workspace: header | counts | order | lists.
struct AttnWs {
    WsHeader* hdr;
    int32_t* counts;   // [B,H,nqb]   number of listed key blocks of each query block
    int32_t* order;    // [B,H,nqb]   query blocks of a head, longest list first
    int32_t* lists;    // [B,H,nqb,nkb] ascending key-block indices, first counts[...] entries valid
    size_t bytes;
};

inline AttnWs attn_ws_layout(void* base, int B, int H, int nqb, int nkb) {
    AttnWs w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.hdr = reinterpret_cast<WsHeader*>(p + off);           off += align256(sizeof(WsHeader));
    size_t rows = size_t(B) * H * nqb;
    w.counts = reinterpret_cast<int32_t*>(p + off);         off += align256(rows * 4);
    w.order = reinterpret_cast<int32_t*>(p + off);          off += align256(rows * 4);
    w.lists = reinterpret_cast<int32_t*>(p + off);          off += align256(rows * size_t(nkb) * 4);
    w.bytes = off;
    return w;
}

// Layout of the builder workspace: header | pooled-blocks counters | qbar | kbar | scores | three-term means of Q, of K.
struct BuildWs {
    WsHeader* hdr;
    int32_t* done;   // [B,H]  pooled blocks of each head written so far (fused builder; zeroed together with the header)
    float* qbar;     // [B,H,nqb,D]
    float* kbar;     // [B,H,nkb,D]
    float* scores;   // [B,H,nqb,nkb]
    __nv_bfloat16* qsplit;   // [3][B*H*nqb][D]  block means of Q as three bf16 terms (fused builder)
    __nv_bfloat16* ksplit;   // [3][B*H*nkb][D]
    size_t bytes;
};

inline BuildWs build_ws_layout(void* base, int B, int H, int nqb, int nkb, int D) {
    BuildWs w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.hdr = reinterpret_cast<WsHeader*>(p + off);           off += align256(sizeof(WsHeader));
    w.done = reinterpret_cast<int32_t*>(p + off);           off += align256(size_t(B) * H * 4);
    w.qbar = reinterpret_cast<float*>(p + off);             off += align256(size_t(B) * H * nqb * D * 4);
    w.kbar = reinterpret_cast<float*>(p + off);             off += align256(size_t(B) * H * nkb * D * 4);
    w.scores = reinterpret_cast<float*>(p + off);           off += align256(size_t(B) * H * nqb * size_t(nkb) * 4);
    w.qsplit = reinterpret_cast<__nv_bfloat16*>(p + off);   off += align256(size_t(3) * B * H * nqb * D * 2);
    w.ksplit = reinterpret_cast<__nv_bfloat16*>(p + off);   off += align256(size_t(3) * B * H * nkb * D * 2);
    w.bytes = off;
    return w;
}

__device__ inline void set_status(WsHeader* hdr, int32_t code, int32_t i0, int32_t i1, int32_t i2) {
    if (atomicCAS(&hdr->status, 0, code) == 0) {
        hdr->info[0] = i0; hdr->info[1] = i1; hdr->info[2] = i2;
    }
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Token geometry used by the always-kept rule of the builder.
struct Geometry {
    int N, n_text, hw, T, bq, bk, window, text_dense;
};

}  // namespace carnator
