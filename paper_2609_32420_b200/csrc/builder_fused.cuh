// M1 + M2 + M3 of the connectivity builder in one persistent kernel (top-k mode, nkb <= 1024): one CTA per SM,
// warp-specialised, so that the fp32 scoring and the selection run underneath the HBM-bound pooling and the pooled
// scores never make the round trip through HBM.
// Paper: Appendix "Reuse-Scope Implementation Details" (per head and query block, the smallest set of key blocks
// covering a fixed fraction of the attention mass), in the pooled-score form.
//
//   warps 0-3   pooling epilogue: one thread per head-dimension element reads its column sum from tensor memory,
//               divides by the number of valid tokens and writes the fp32 block mean
//   warp 4      pooling producer (one lane): takes (head, tensor, block) items from a counter and brings each block
//               into a shared-memory ring with TMA (and asks L2 for blocks further ahead)
//   warp 5      pooling sums on the tensor cores (one lane): sum over tokens = X^T (the block as an MN-major A
//               operand, one row per head-dimension element) times a 128 x 16 matrix of ones, fp32 accumulate in
//               tensor memory; the CUDA cores then only touch D values per block, which leaves the issue slots of
//               the SM to the scoring group
//   warps 8-23  scoring group: takes (head, R query blocks) items from a second counter, waits (bounded) until the
//               head's pooled vectors are complete, computes its R x nkb fp32 pooled scores (plain FFMA, key blocks
//               streamed through shared memory from L2) into shared memory, and selects per row with the keys in
//               registers as select_topk_kernel does; only the uint8 mask (and the scores, if the caller asked for
//               them) goes to global memory
// Items are taken in head order, so scoring of head h runs under the pooling of head h + 1.  A scoring item only
// waits for pooling items that were taken before it, and the pooling warps wait only for one another, so the waits
// always end; every wait is bounded all the same.
#pragma once
#include "builder.cuh"
#include "attn_tcgen05.cuh"

namespace carnator {

constexpr int kFusedPoolThreads = 256;      // warps 0-7 (two warpgroups, so that registers can move: warps 6 and 7 idle)
constexpr int kFusedScoreThreads = 512;     // warps 8-23
constexpr int kFusedThreads = kFusedPoolThreads + kFusedScoreThreads;
constexpr int kFusedStages = 4;       // blocks in the pooling ring
constexpr int kFusedBatch = 4;        // pooling items taken per counter update; L2 is asked for one batch ahead
constexpr int kFusedQueue = 8;        // decoded items in flight between producer and epilogue (> kFusedStages + 2)
constexpr int kFusedRows = 32;        // query blocks per scoring item (two per warp of the scoring group)
constexpr int kFusedCols = 256;       // key blocks per score tile
constexpr int kFusedSlab = 16;        // head-dimension slab per shared-memory stage

struct FusedArgs {
    PoolArgs pool;
    SelectArgs sel;
    float* scores_out;      // [B,H,nqb,nkb] or nullptr
    int32_t* done;          // [B,H]
    WsHeader* hdr;
    int B;
    float scale;
};

struct PoolItem {           // one decoded pooling item, producer -> epilogue
    float* dst;             // where the D means go (nullptr: end marker)
    int nvalid, bh, block;  // valid tokens, head, token rows of the tile
};

__device__ __forceinline__ void named_bar(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ float tmem_ld1(uint32_t taddr) {
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
    return __uint_as_float(r);
}

// TR consecutive floats from shared memory in one load (the address is a multiple of 4 * TR bytes)
template <int TR>
__device__ __forceinline__ void load_rows(float (&ar)[TR], const float* p) {
    if constexpr (TR == 4) { const float4 v = *reinterpret_cast<const float4*>(p); ar[0] = v.x; ar[1] = v.y; ar[2] = v.z; ar[3] = v.w; }
    else if constexpr (TR == 2) { const float2 v = *reinterpret_cast<const float2*>(p); ar[0] = v.x; ar[1] = v.y; }
    else { ar[0] = p[0]; }
}

template <int D, int R>
struct FusedSmem {
    static constexpr size_t kBox = size_t(128) * 128;                             // 128 token rows x 64 elements, 128-byte swizzle
    static constexpr size_t kSlot = (D / 64) * kBox;                              // one block of up to 128 tokens
    static constexpr size_t kOffRing = 0;                                         // 1 KiB aligned
    static constexpr size_t kOffOnes = kOffRing + kFusedStages * kSlot;           // 16 rows x 128 B of bf16 ones (B operand)
    static constexpr size_t kOffBar = kOffOnes + 2048;                            // mbarriers
    static constexpr size_t kOffA = kOffBar + 256;                                // [D][R + 4]
    static constexpr size_t kOffB = kOffA + size_t(D) * (R + 4) * 4;              // [2][kFusedSlab][kFusedCols + 4]
    static constexpr size_t kOffFrames = kOffB + 2 * size_t(kFusedSlab) * (kFusedCols + 4) * 4; // int2 [nkb]
    static size_t bytes(int nkb) { return kOffFrames + size_t(nkb) * 8 + 1024; }   // + slack to align the base
};

template <int D, int NPL, int R>
__global__ void __launch_bounds__(kFusedThreads, 1)
build_fused_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK, const FusedArgs a) {
    extern __shared__ unsigned char fsm_raw[];
    __shared__ PoolItem pool_q[kFusedQueue];
    __shared__ int score_item[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    using L = FusedSmem<D, R>;
    const int tid = threadIdx.x, warp_id = tid >> 5, lane = tid & 31;
    const int nqb = a.sel.nqb, nkb = a.sel.nkb, H = a.sel.H;
    const int heads = a.B * H;
    const uint32_t smem_base = (smem_u32(fsm_raw) + 1023u) & ~1023u;
    unsigned char* fsm = fsm_raw + (smem_base - smem_u32(fsm_raw));
    const uint32_t bars = smem_base + uint32_t(L::kOffBar);
    auto bar_full = [&](int s) { return bars + 8 * s; };             // block s of the ring has landed
    auto bar_empty = [&](int s) { return bars + 32 + 8 * s; };       // the sums of the block in slot s are done
    auto bar_acc = [&](int s) { return bars + 64 + 8 * s; };         // accumulator s holds fresh sums
    auto bar_accfree = [&](int s) { return bars + 80 + 8 * s; };     // the epilogue has read accumulator s
    const uint32_t bar_drain = bars + 96;
    volatile int* abortp = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kFusedStages; ++s) { tc::mbar_init(bar_full(s), 1); tc::mbar_init(bar_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { tc::mbar_init(bar_acc(s), 1); tc::mbar_init(bar_accfree(s), 4); }
        tc::mbar_init(bar_drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 2048 / 4) reinterpret_cast<uint32_t*>(fsm + L::kOffOnes)[tid] = 0x3F803F80u;      // bf16 1.0 pairs
    if (warp_id == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(32) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the ones are read by the tensor cores (async proxy)
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const int per_head = nqb + nkb;
    const int pool_total = heads * per_head;

    // Register budget: 768 threads x 80 at launch; the pooling warps keep 32 each, the scoring group takes 104
    // (256 x 32 + 512 x 104 = 768 x 80), enough to hold two rows of scores per warp.
    if (warp_id < 8) asm volatile("setmaxnreg.dec.sync.aligned.u32 32;" ::: "memory");
    if (warp_id < 4) {
        // ================= pooling epilogue: tensor memory -> block means =================
        const int d = warp_id * 32 + lane;                             // head-dimension element = tensor-memory lane
        const uint32_t lane_base = uint32_t(warp_id * 32) << 16;
        int pub_count = 0, pub_head = -1;
        bool ok = true;
        for (int n = 0; ok; ++n) {
            const int buf = n & 1;
            ok = tc::mbar_wait_warp(bar_acc(buf), uint32_t(n >> 1) & 1u, abortp, 64);
            if (!ok) { if (lane == 0 && !*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 41, n, blockIdx.x); break; }
            const PoolItem it = pool_q[n % kFusedQueue];
            if (it.dst == nullptr) break;                              // the producer's end marker
            tc::tc_fence_after();
            const float sum = tmem_ld1(tmem + lane_base + uint32_t(buf * 16));
            tc::tmem_wait_ld();
            tc::tc_fence_before();
            tc::mbar_arrive_warp(bar_accfree(buf));
            if (d < D) it.dst[d] = sum / float(it.nvalid);
            // A head's counter moves when this CTA leaves the head (one fence per head, not one per block).  The named
            // barrier orders the four warps' stores before thread 0's fence.
            named_bar(1, 128);
            if (tid == 0) {
                if (it.bh != pub_head && pub_count > 0) { __threadfence(); atomicAdd(&a.done[pub_head], pub_count); pub_count = 0; }
                pub_head = it.bh;
                ++pub_count;
            }
        }
        named_bar(1, 128);
        if (tid == 0 && pub_count > 0) { __threadfence(); atomicAdd(&a.done[pub_head], pub_count); }
    } else if (warp_id == 4) {
        // ================= pooling producer =================
        if (lane == 0) {
            tc::prefetch_tmap(&mapQ); tc::prefetch_tmap(&mapK);
            // item number -> tensor-map coordinates; K blocks of a head first, then its Q blocks
            auto coords = [&](int item, int& which, int& I, int& h, int& b) {
                const int bh = item / per_head, rem = item - bh * per_head;
                which = rem < nkb ? 1 : 0;
                I = which ? rem : rem - nkb;
                b = bh / H; h = bh - b * H;
                return bh;
            };
            // Items are taken four at a time (one counter update per four blocks; consecutive blocks also sit next to
            // each other in HBM).  While one batch is loaded, L2 is asked for the whole next batch.
            auto prefetch_batch = [&](int base) {
                for (int j = 0; j < kFusedBatch; ++j) {
                    if (base + j >= pool_total) break;
                    int which, I, h, b; coords(base + j, which, I, h, b);
                    const int block = which ? a.pool.block[1] : a.pool.block[0];
#pragma unroll
                    for (int x = 0; x < D / 64; ++x) tma_prefetch_4d(which ? &mapK : &mapQ, x * 64, I * block, h, b);
                }
            };
            int base_cur = atomicAdd(&a.hdr->work[0], kFusedBatch);
            int base_next = atomicAdd(&a.hdr->work[0], kFusedBatch);
            prefetch_batch(base_cur);
            int armed = -1, n = 0;
            bool more = true;
            while (more) {
                prefetch_batch(base_next);
                const int base_after = atomicAdd(&a.hdr->work[0], kFusedBatch);      // needed one batch from now: its latency hides
                for (int j = 0; j < kFusedBatch; ++j, ++n) {
                    const int item = base_cur + j;
                    const int s = n % kFusedStages;
                    PoolItem it; it.dst = nullptr; it.nvalid = 0; it.bh = -1; it.block = 0;
                    if (n >= kFusedStages && !tc::mbar_wait(bar_empty(s), uint32_t(n / kFusedStages - 1) & 1u, abortp, 64)) {
                        if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 42, n, blockIdx.x);
                        *abortp = 1; more = false; break;
                    }
                    if (item >= pool_total) {                          // end marker for the MMA warp and the epilogue
                        pool_q[n % kFusedQueue] = it;
                        tc::mbar_arrive(bar_full(s));
                        more = false; break;
                    }
                    int which, I, h, b;
                    const int bh = coords(item, which, I, h, b);
                    const int block = which ? a.pool.block[1] : a.pool.block[0];
                    it.dst = (which ? a.pool.out[1] : a.pool.out[0]) + (int64_t(bh) * (which ? nkb : nqb) + I) * D;
                    it.nvalid = min(block, a.pool.N - I * block);
                    it.bh = bh; it.block = block;
                    pool_q[n % kFusedQueue] = it;                      // read by the others only after bar_full / bar_acc of this item
                    tc::mbar_expect_tx(bar_full(s), uint32_t(block) * D * 2);
#pragma unroll
                    for (int x = 0; x < D / 64; ++x)
                        tc::tma_load_4d(smem_base + uint32_t(L::kOffRing + s * L::kSlot + x * L::kBox), which ? &mapK : &mapQ,
                                        bar_full(s), x * 64, I * block, h, b);
                    armed = n;
                }
                base_cur = base_next; base_next = base_after;
            }
            if (*abortp)       // copies in flight must land before the CTA gives its shared memory back
                for (int k = 0; k < kFusedStages && armed - k >= 0; ++k)
                    tc::mbar_wait_drain(bar_full((armed - k) % kFusedStages), uint32_t((armed - k) / kFusedStages) & 1u);
        }
    } else if (warp_id == 5) {
        // ================= pooling sums on the tensor cores =================
        if (lane == 0) {
            // A = the block, MN-major (rows = head-dimension elements, 64-element chunks one box apart; for D = 64 the
            // upper 64 rows of the 128-row product repeat the lower ones and are never read); B = ones, K-major.
            constexpr uint32_t idesc = tc::instr_desc(128, 16, 0) | (1u << 15);
            const uint64_t da0 = tc::smem_desc(smem_base + uint32_t(L::kOffRing), D == 128 ? uint32_t(L::kBox) : 0u, 1024);
            const uint64_t db = tc::smem_desc(smem_base + uint32_t(L::kOffOnes), 16, 1024);
            bool ok = true;
            for (int n = 0; ok; ++n) {
                const int s = n % kFusedStages, buf = n & 1;
                ok = tc::mbar_wait(bar_full(s), uint32_t(n / kFusedStages) & 1u, abortp, 32);
                if (!ok) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 43, n, blockIdx.x); *abortp = 1; break; }
                const PoolItem it = pool_q[n % kFusedQueue];
                if (n >= 2) {
                    ok = tc::mbar_wait(bar_accfree(buf), uint32_t((n - 2) >> 1) & 1u, abortp, 32);
                    if (!ok) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 44, n, blockIdx.x); *abortp = 1; break; }
                }
                if (it.dst == nullptr) { tc::mbar_arrive(bar_acc(buf)); break; }      // pass the end marker on
                tc::tc_fence_after();
                const int ksteps = (it.block + 15) / 16;                              // token rows past the valid ones read as zero
                const uint64_t da = da0 + uint64_t((uint32_t(s) * uint32_t(L::kSlot)) >> 4);
                for (int kk = 0; kk < ksteps; ++kk)
                    tc::mma_ss(tmem + uint32_t(buf * 16), da + uint64_t(kk * (2048 >> 4)), db, idesc, kk > 0 ? 1u : 0u);
                tc::tc_commit(bar_acc(buf));
                tc::tc_commit(bar_empty(s));
            }
            tc::tc_commit(bar_drain);                                  // no product may still run when tensor memory is released
            tc::mbar_wait_drain(bar_drain, 0);
        }
    } else if (warp_id >= 8) {
    // ================= scoring + selection group =================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 104;" ::: "memory");
    const int t = tid - kFusedPoolThreads;
    constexpr int NT = kFusedScoreThreads;
    constexpr int NW = NT / 32;                                        // 16 warps
    constexpr int RS = R / NW;                                         // query blocks (rows) per warp: scored and selected in registers
    static_assert(RS == 1 || RS == 2, "rows per scoring item");
    static_assert(NPL % 8 == 0, "a lane holds eight columns per tile");
    float* sA = reinterpret_cast<float*>(fsm + L::kOffA);            // [D][R + 4]   q_bar of the item, k-major
    float* sB = reinterpret_cast<float*>(fsm + L::kOffB);            // [2][kFusedSlab][kFusedCols + 4]
    int2* kframes = reinterpret_cast<int2*>(fsm + L::kOffFrames);
    constexpr int LDA = R + 4, LDB = kFusedCols + 4;
    const Geometry g = a.sel.g;
    for (int J = t; J < nkb; J += NT) {
        const int k_lo = max(J * g.bk, g.n_text), k_hi = min(g.N, (J + 1) * g.bk) - 1;
        kframes[J] = (k_hi >= k_lo) ? make_int2((k_lo - g.n_text) / g.hw, (k_hi - g.n_text) / g.hw) : make_int2(1, 0);
    }
    const int groups_per_head = (nqb + R - 1) / R;
    const int total = heads * groups_per_head;
    const int warp = t >> 5;
    const int r0 = warp * RS;                                          // this warp's rows of the item
    const int text_cols = (g.text_dense && g.n_text > 0) ? (g.n_text + g.bk - 1) / g.bk : 0;
    const int ntiles = (nkb + kFusedCols - 1) / kFusedCols;
    const int nslabs = ntiles * (D / kFusedSlab);
    // loader mapping of a 256-column x 16 slab: thread -> key blocks (t / 4) and (t / 4) + 128, four of the 16 k (64
    // contiguous bytes per key block per slab).  Lane l scores columns l, l + 32, ..., l + 224; in a shared-memory row
    // its first four sit at 4 l .. 4 l + 3 and its last four at 128 + 4 l .., so a warp's 16-byte loads are contiguous.
    const int lcol = t >> 2, lk = (t & 3) * 4;
    const int lpos0 = (lcol & 31) * 4 + (lcol >> 5), lpos1 = lpos0 + 128;
    int ready_head = -1;
    for (;;) {
        named_bar(2, NT);                                             // previous item's shared memory is no longer read
        if (t == 0) score_item[0] = atomicAdd(&a.hdr->work[1], 1);
        named_bar(2, NT);
        const int item = score_item[0];
        if (item >= total) break;
        const int bh = item / groups_per_head;
        const int I0 = (item % groups_per_head) * R;
        const int nrows = min(R, nqb - I0);
        if (bh != ready_head) {                                        // the head's pooled vectors must all be written
            if (t == 0) {
                int ok = 1;
                if (ld_acquire(a.done + bh) < nqb + nkb) {
                    const unsigned long long t0 = global_timer_ns();
                    ok = 0;
                    for (uint32_t it = 0; it < (1u << 30); ++it) {
                        __nanosleep(200);
                        if (ld_acquire(a.done + bh) >= nqb + nkb) { ok = 1; break; }
                        if ((it & 63u) == 63u && (*abortp || global_timer_ns() - t0 > 2000000000ull)) break;
                    }
                }
                if (!ok) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 40, bh, blockIdx.x);
                score_item[1] = ok;
            }
            named_bar(2, NT);
            if (!score_item[1]) break;
            ready_head = bh;
        }
        const float* qb = a.pool.out[0] + (int64_t(bh) * nqb + I0) * D;
        const float* kb = a.pool.out[1] + int64_t(bh) * nkb * D;
        // q_bar of the item, transposed to k-major (rows past the head's last query block read as zero)
        for (int idx = t; idx < R * (D / 4); idx += NT) {
            const int row = idx % R, k4 = (idx / R) * 4;               // consecutive threads -> consecutive rows: conflict-free stores
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < nrows) v = __ldcg(reinterpret_cast<const float4*>(qb + int64_t(row) * D + k4));
            sA[(k4 + 0) * LDA + row] = v.x; sA[(k4 + 1) * LDA + row] = v.y;
            sA[(k4 + 2) * LDA + row] = v.z; sA[(k4 + 3) * LDA + row] = v.w;
        }
        // ---- scores: the pooled vectors of the key blocks stream through a double-buffered slab, one barrier per slab;
        //      every warp keeps the scores of its rows in registers, in the layout the selection wants ----
        uint32_t key[RS][NPL];                                        // first the fp32 scores (as bits), then their order-preserving keys
#pragma unroll
        for (int i = 0; i < RS; ++i)
#pragma unroll
            for (int q = 0; q < NPL; ++q) key[i][q] = 0u;
        float4 pre[2];
        auto fetch = [&](int slab) {
            const int j0 = (slab / (D / kFusedSlab)) * kFusedCols, k0 = (slab % (D / kFusedSlab)) * kFusedSlab;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int col = j0 + lcol + q * 128;
                pre[q] = (col < nkb) ? __ldcg(reinterpret_cast<const float4*>(kb + int64_t(col) * D + k0 + lk)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        };
        auto stash = [&](int buf) {
            float* dst = sB + buf * (kFusedSlab * LDB) + lk * LDB;
            dst[0 * LDB + lpos0] = pre[0].x; dst[1 * LDB + lpos0] = pre[0].y; dst[2 * LDB + lpos0] = pre[0].z; dst[3 * LDB + lpos0] = pre[0].w;
            dst[0 * LDB + lpos1] = pre[1].x; dst[1 * LDB + lpos1] = pre[1].y; dst[2 * LDB + lpos1] = pre[1].z; dst[3 * LDB + lpos1] = pre[1].w;
        };
        fetch(0);
        stash(0);
        named_bar(2, NT);                                              // slab 0 and sA are in place
        float acc[RS][8];
#pragma unroll 1
        for (int slab = 0; slab < nslabs; ++slab) {
            const int tile = slab / (D / kFusedSlab), k0 = (slab % (D / kFusedSlab)) * kFusedSlab;
            if (slab + 1 < nslabs) fetch(slab + 1);
            if (k0 == 0) {
#pragma unroll
                for (int i = 0; i < RS; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
            }
            const float* bs = sB + (slab & 1) * (kFusedSlab * LDB) + lane * 4;
            const float* as = sA + k0 * LDA + r0;
            const bool upper = tile * kFusedCols + 128 < nkb;          // warp-uniform: columns 128.. of this tile hold key blocks
            if (upper) {
#pragma unroll
                for (int k = 0; k < kFusedSlab; ++k) {
                    float ar[RS];
                    load_rows<RS>(ar, as + k * LDA);
                    const float4 b0 = *reinterpret_cast<const float4*>(bs + k * LDB);
                    const float4 b1 = *reinterpret_cast<const float4*>(bs + k * LDB + 128);
                    const float br[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                    for (int i = 0; i < RS; ++i)
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
                }
            } else {
#pragma unroll
                for (int k = 0; k < kFusedSlab; ++k) {
                    float ar[RS];
                    load_rows<RS>(ar, as + k * LDA);
                    const float4 b0 = *reinterpret_cast<const float4*>(bs + k * LDB);
                    const float br[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
                    for (int i = 0; i < RS; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
                }
            }
            if (k0 + kFusedSlab == D) {                                 // the tile is complete: its scores move to their place
#pragma unroll
                for (int tt = 0; tt < NPL / 8; ++tt)
                    if (tt == tile) {
#pragma unroll
                        for (int i = 0; i < RS; ++i)
#pragma unroll
                            for (int j = 0; j < 8; ++j) key[i][tt * 8 + j] = __float_as_uint(a.scale * acc[i][j]);
                    }
            }
            if (slab + 1 < nslabs) stash((slab + 1) & 1);
            named_bar(2, NT);
        }
        // ---- selection: each warp on its own rows (two independent rows fill each other's latencies) ----
        {
            uint32_t forced_bits[RS][(NPL + 31) / 32];
            int n_admit[RS];
#pragma unroll
            for (int i = 0; i < RS; ++i) {
                const int rr = r0 + i;
                const int I = I0 + rr;
                const int64_t row = (int64_t(bh) * nqb + I) * nkb;
                const bool live = rr < nrows;                           // warp-uniform
                const bool text_row = g.text_dense && g.n_text > 0 && I * g.bq < g.n_text;
                int f_lo = 0, f_hi = 0;
                bool has_window = false;
                if (g.window >= 0) {
                    const int q_lo = max(I * g.bq, g.n_text), q_hi = min(g.N, (I + 1) * g.bq) - 1;
                    if (q_hi >= q_lo) {
                        has_window = true;
                        f_lo = max(0, (q_lo - g.n_text) / g.hw - g.window);
                        f_hi = min(g.T - 1, (q_hi - g.n_text) / g.hw + g.window);
                    }
                }
#pragma unroll
                for (int w = 0; w < (NPL + 31) / 32; ++w) forced_bits[i][w] = 0u;
                int my_forced = 0;
#pragma unroll
                for (int q = 0; q < NPL; ++q) {
                    const int J = q * 32 + lane;
                    uint32_t k = 0u;                                    // always-kept and out-of-range entries never compete
                    if (live && J < nkb) {
                        const float v = __uint_as_float(key[i][q]);
                        const int2 kf = kframes[J];
                        const bool forced = text_row || J < text_cols || (has_window && kf.x <= kf.y && kf.x <= f_hi && kf.y >= f_lo);
                        if (forced) { forced_bits[i][q >> 5] |= 1u << (q & 31); ++my_forced; }
                        else k = ordered_bits(v);
                        if (a.scores_out) a.scores_out[row + J] = v;
                    }
                    key[i][q] = k;
                }
                const int nforced = __reduce_add_sync(0xffffffffu, my_forced);
                const int nfree = nkb - nforced;
                int na = a.sel.count_includes_forced ? max(0, a.sel.k_all - nforced) : topk_count_dev(a.sel.keep_ratio, nfree);
                n_admit[i] = live ? min(na, nfree) : 0;
            }
            // k-th largest key of every row, bit by bit: the largest T with #(key >= T) >= n_admit.  Once a candidate is
            // met by exactly n_admit keys the kept set is known (the remaining bits would only find its smallest key).
            uint32_t T[RS];
            bool exact[RS];
#pragma unroll
            for (int i = 0; i < RS; ++i) { T[i] = 0u; exact[i] = n_admit[i] == 0; }
#pragma unroll 1
            for (int bit = 31; bit >= 0; --bit) {
                bool all_exact = true;
#pragma unroll
                for (int i = 0; i < RS; ++i) all_exact = all_exact && exact[i];
                if (all_exact) break;                                   // warp-uniform
                int cnt[RS];
#pragma unroll
                for (int i = 0; i < RS; ++i) {
                    const uint32_t cand = T[i] | (1u << bit);
                    int c0 = 0, c1 = 0;
#pragma unroll
                    for (int q = 0; q + 1 < NPL; q += 2) { c0 += (key[i][q] >= cand) ? 1 : 0; c1 += (key[i][q + 1] >= cand) ? 1 : 0; }
                    cnt[i] = c0 + c1;
                }
#pragma unroll
                for (int i = 0; i < RS; ++i) {
                    const int c = __reduce_add_sync(0xffffffffu, cnt[i]);
                    if (!exact[i] && c >= n_admit[i]) { T[i] |= (1u << bit); exact[i] = (c == n_admit[i]); }
                }
            }
#pragma unroll
            for (int i = 0; i < RS; ++i) {
                const int rr = r0 + i;
                if (rr >= nrows) continue;                              // warp-uniform
                const int64_t row = (int64_t(bh) * nqb + I0 + rr) * nkb;
                const bool any = n_admit[i] > 0;                        // n_admit == 0: nothing is admitted by score
                int gt = 0;
#pragma unroll
                for (int q = 0; q < NPL; ++q) gt += (key[i][q] > T[i]) ? 1 : 0;
                gt = __reduce_add_sync(0xffffffffu, gt);
                const int need_eq = n_admit[i] - gt;                    // blocks with key == T, lowest block index first
                int seen_eq = 0;
#pragma unroll
                for (int q = 0; q < NPL; ++q) {
                    const int J = q * 32 + lane;
                    const bool eq = any && key[i][q] == T[i];
                    const unsigned bal = __ballot_sync(0xffffffffu, eq);
                    const int rank = seen_eq + __popc(bal & ((1u << lane) - 1u));
                    seen_eq += __popc(bal);
                    const bool keep = ((forced_bits[i][q >> 5] >> (q & 31)) & 1u) || (any && key[i][q] > T[i]) || (eq && rank < need_eq);
                    if (J < nkb) a.sel.mask[row + J] = keep ? 1 : 0;
                }
            }
        }
    }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp_id == 5) {
        tc::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(32) : "memory");
    }
}

}  // namespace carnator
