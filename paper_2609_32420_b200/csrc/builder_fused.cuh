// M1 + M2 + M3 of the connectivity builder in one persistent kernel (top-k mode, nkb <= 1024): one CTA per SM,
// warp-specialised, so that scoring and selection run underneath the HBM-bound pooling and the pooled scores never
// make the round trip through HBM.
// Paper: Appendix "Reuse-Scope Implementation Details" (per head and query block, the smallest set of key blocks
// covering a fixed fraction of the attention mass), in the pooled-score form.
//
//   warps 0-3   pooling epilogue: one thread per head-dimension element reads its column sum from tensor memory,
//               divides by the number of valid tokens and writes the block mean as three bf16 terms
//               (mean = t1 + t2 + t3 to fp32 precision)
//   warp 4      pooling producer (one lane): takes (head, tensor, block) items from a counter and brings each block
//               into a shared-memory ring with TMA (and asks L2 for blocks further ahead); at D = 64 an item is two
//               consecutive blocks, which fill the 128 rows of the product as the two halves of a D = 128 block do
//   warp 5      pooling sums on the tensor cores (one lane): sum over tokens = X^T (the block as an MN-major A
//               operand, one row per head-dimension element) times a 128 x 16 matrix of ones, fp32 accumulate in
//               tensor memory; the CUDA cores then only touch D values per block
//   warp 6      score producer (one lane): takes (head, 16 query blocks) items from a second counter, waits (bounded)
//               until the head's pooled vectors are complete, and brings their three-term forms in with TMA
//   warp 7      scores on the tensor cores (one lane): S^T[J, I] = sum_d k_bar[J, d] q_bar[I, d] as six bf16 products
//               (t1 t1, t1 t2, t2 t1, t1 t3, t2 t2, t3 t1: what is left out is below 2^-24 of the score), fp32
//               accumulate in tensor memory (the large product and the small ones apart), 128 key blocks x 16 query
//               blocks per instruction
//   warps 8-23  selection group: moves the scores of an item from tensor memory into shared memory rows (one row per
//               query block), then each warp selects for one row with the keys in registers, as select_topk_kernel
//               does; only the uint8 mask (and the scores, if the caller asked for them) goes to global memory
// Items are taken in head order, so scoring of head h runs under the pooling of head h + 1.  A scoring item only
// waits for pooling items that were taken before it, and the pooling warps wait only for one another, so the waits
// always end; every wait is bounded all the same.
#pragma once
#include "builder.cuh"
#include "attn_tcgen05.cuh"

namespace carnator {

constexpr int kFusedPoolThreads = 256;      // warps 0-7: pooling (0-5) and score operands / products (6-7)
constexpr int kFusedScoreThreads = 512;     // warps 8-23: selection group
constexpr int kFusedThreads = kFusedPoolThreads + kFusedScoreThreads;
// blocks in the pooling ring (PST: 3, or 2 where the score rows of a long layer need the room) and buffers of the
// key-block operand of the score products (AST: 3 where they fit, else 2) are template parameters of the kernel
constexpr int kFusedBatchBytes = 64 * 1024;    // consecutive bytes of Q or K a CTA takes per counter update (2 or 4 blocks)
constexpr int kFusedAheadBytes = 128 * 1024;   // how far ahead of the loads L2 is asked for the blocks to come
constexpr int kFusedQueue = 8;        // decoded items in flight between producer and epilogue (> PST + 2)
constexpr int kFusedRows = 16;        // query blocks per scoring item (N of the score products; one selection warp each)
constexpr int kFusedTmemCols = 512;   // [0, 32): two pooling accumulators; [32, 512): score tiles

struct FusedArgs {
    PoolArgs pool;
    SelectArgs sel;
    float* scores_out;      // [B,H,nqb,nkb] or nullptr
    __nv_bfloat16* split[2];   // [3][B*H*nb][D]: the three bf16 terms of the block means of Q (0) and K (1)
    int32_t* done;          // [B,H]
    WsHeader* hdr;
    int B;
    float scale;
    int nkb_pad;            // row stride of the shared-memory score rows (floats)
};

struct __align__(16) PoolItem {   // one pooling item, producer -> MMA warp and epilogue (16 bytes: one shared-memory store)
    int bh;                 // head (batch-major); < 0: end marker
    int I;                  // (first) block index, bit 30 set for a K block
    int block, nvalid;      // token rows of the tile, valid tokens among them
};
struct ScoreItem { int bh, I0; };     // bh < 0: end marker

// tcgen05.mma with both operands in shared memory, for a converged warp: every lane executes the statement with the same
// operands and one elected lane issues (the compiler keeps the descriptors in uniform registers, and the warp spends far
// fewer issue slots per instruction than a single lane inside a branch does)
__device__ __forceinline__ void mma_ss_elect(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void named_bar(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void tma_prefetch_5d(const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4) {
    asm volatile("cp.async.bulk.prefetch.tensor.5d.L2.global.tile [%0, {%1, %2, %3, %4, %5}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ float tmem_ld1(uint32_t taddr) {
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
    return __uint_as_float(r);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory plan.  Pooling ring: blocks of 128 token rows as D/64 boxes (128 rows x 128 B, 128-byte swizzle).
// Score operands: A = the three terms of 128 key-block means, one 32-element quarter of the head dimension at a time
// (3 boxes of 128 rows x 64 B, 64-byte swizzle), AST buffers; B = the three terms of the item's 16 query-block means,
// whole rows (boxes of 16 rows x 128 B, 128-byte swizzle).
template <int D, int PST, int AST>
struct FusedSmem {
    static constexpr size_t kBox = size_t(128) * 128;
    static constexpr size_t kBoxB = size_t(kFusedRows) * 128;                     // 16 query blocks x 64 elements
    static constexpr size_t kSlot = 2 * kBox;                                    // D = 128: the two halves of a block; D = 64: two blocks
    static constexpr size_t kOffRing = 0;                                         // 1 KiB aligned
    static constexpr size_t kBoxA = size_t(128) * 64;                             // 128 key blocks x 32 elements, 64-byte swizzle
    static constexpr size_t kOffScoreA = kOffRing + PST * kSlot;                  // AST buffers x 3 terms x 8 KiB
    static constexpr size_t kOffScoreB = kOffScoreA + AST * 3 * kBoxA;            // 3 terms x D/64 halves x 2 KiB
    static constexpr size_t kOffOnes = kOffScoreB + 3 * (D / 64) * kBoxB;         // 16 rows x 128 B of bf16 ones
    static constexpr size_t kOffBar = kOffOnes + 2048;                            // mbarriers
    static constexpr size_t kOffScores = kOffBar + 256;                           // float [RP][nkb_pad]
    __host__ __device__ static size_t off_scores(int) { return kOffScores; }
    static size_t bytes(int nkb, int nkb_pad) { return off_scores(nkb) + size_t(kFusedRows) * nkb_pad * 4 + 1024; }   // + slack to align the base
};

template <int D, int NPL, int PST, int AST>
__global__ void __launch_bounds__(kFusedThreads, 1)
build_fused_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                   const __grid_constant__ CUtensorMap mapQs, const __grid_constant__ CUtensorMap mapKs, const FusedArgs a) {
    extern __shared__ unsigned char fsm_raw[];
    __shared__ PoolItem pool_q[kFusedQueue];
    __shared__ int ahead_q[8 * 5];                      // the pooling producer's batches taken from the counter and not yet loaded
    __shared__ ScoreItem score_q[4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    constexpr int NR = kFusedRows, RP = kFusedRows;                 // query blocks per item = rows selected at once
    constexpr int kBatch = kFusedBatchBytes / int(FusedSmem<D, PST, AST>::kSlot);   // pooling items per counter update (2)
    // A pooling item fills the 128 rows of the tensor-core product: at D = 128 one block (its two 64-element halves), at
    // D = 64 two consecutive blocks of the same tensor and head.
    constexpr int PB = D == 64 ? 2 : 1;
    using L = FusedSmem<D, PST, AST>;
    constexpr int KH = D / 64;                                         // 64-element halves of the head dimension
    // accumulators per score tile: the large product t1 t1, one per half of the head dimension, apart from the five small ones
    constexpr int NACC = KH + 1;
    const int tid = threadIdx.x, warp_id = tid >> 5, lane = tid & 31;
    const int nqb = a.sel.nqb, nkb = a.sel.nkb, H = a.sel.H;
    const int heads = a.B * H;
    const int ntiles = (nkb + 127) / 128;                              // 128 key blocks per score tile
    const uint32_t smem_base = (smem_u32(fsm_raw) + 1023u) & ~1023u;
    unsigned char* fsm = fsm_raw + (smem_base - smem_u32(fsm_raw));
    const uint32_t bars = smem_base + uint32_t(L::kOffBar);
    auto bar_full = [&](int s) { return bars + 8 * s; };             // block s of the pooling ring has landed
    auto bar_empty = [&](int s) { return bars + 32 + 8 * s; };       // the sums of the block in slot s are done
    auto bar_acc = [&](int s) { return bars + 64 + 8 * s; };         // pooling accumulator s holds fresh sums
    auto bar_accfree = [&](int s) { return bars + 80 + 8 * s; };     // the epilogue has read accumulator s
    const uint32_t bar_drain = bars + 96, bar_drain2 = bars + 104;
    auto bar_afull = [&](int s) { return bars + 160 + 8 * s; };      // score operand A, buffer s (key-block means, one quarter)
    auto bar_afree = [&](int s) { return bars + 192 + 8 * s; };
    const uint32_t bar_bfull = bars + 128, bar_bfree = bars + 136;   // score operand B (the item's query-block means)
    const uint32_t bar_sfull = bars + 144, bar_sfree = bars + 152;   // the item's scores in tensor memory
    volatile int* abortp = &abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < PST; ++s) { tc::mbar_init(bar_full(s), 1); tc::mbar_init(bar_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { tc::mbar_init(bar_acc(s), 1); tc::mbar_init(bar_accfree(s), 4); }
        tc::mbar_init(bar_drain, 1); tc::mbar_init(bar_drain2, 1);
        for (int s = 0; s < AST; ++s) { tc::mbar_init(bar_afull(s), 1); tc::mbar_init(bar_afree(s), 1); }
        tc::mbar_init(bar_bfull, 1); tc::mbar_init(bar_bfree, 1);
        tc::mbar_init(bar_sfull, 1); tc::mbar_init(bar_sfree, kFusedScoreThreads / 32);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 2048 / 4) reinterpret_cast<uint32_t*>(fsm + L::kOffOnes)[tid] = 0x3F803F80u;      // bf16 1.0 pairs
    if (warp_id == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kFusedTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the ones are read by the tensor cores (async proxy)
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tmem_s = tmem + 32;                                // score tiles (behind the two pooling accumulators)
    const int nqi = (nqb + PB - 1) / PB, nki = (nkb + PB - 1) / PB;     // pooling items per head and tensor
    const int per_head = nqi + nki;
    const int pool_total = heads * per_head;
    const int groups_per_head = (nqb + NR - 1) / NR;
    const int score_total = heads * groups_per_head;

    // Register budget: 768 threads x 80 at launch; the pooling and operand warps keep 40 each, the selection group takes
    // 96 (256 x 40 + 512 x 96 <= 768 x 80).
    if (warp_id < 8) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
    if (warp_id < 4) {
        // ================= pooling epilogue: tensor memory -> block means as three bf16 terms =================
        const int r = warp_id * 32 + lane;                             // tensor-memory lane: head-dimension element (and block, D = 64)
        const int d = r & (D - 1);
        const uint32_t lane_base = uint32_t(warp_id * 32) << 16;
        int pub_count = 0, pub_head = -1;
        bool ok = true;
        for (int n = 0; ok; ++n) {
            const int buf = n & 1;
            ok = tc::mbar_wait_warp(bar_acc(buf), uint32_t(n >> 1) & 1u, abortp, 64);
            if (!ok) { if (lane == 0 && !*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 41, n, blockIdx.x); break; }
            const PoolItem it = pool_q[n % kFusedQueue];
            if (it.bh < 0) break;                                      // the producer's end marker
            // where the three terms go (this warp has time to spare; the producer thread does not)
            const int which = it.I >> 30, nb = which ? nkb : nqb;
            const int I = (it.I & 0x3FFFFFFF) + r / D;                  // this lane's block (D = 64: lanes 64-127 hold the item's second block)
            __nv_bfloat16* const dst = a.split[which] + (int64_t(it.bh) * nb + I) * D;
            const int64_t term_stride = int64_t(heads) * nb * D;
            tc::tc_fence_after();
            const float sum = tmem_ld1(tmem + lane_base + uint32_t(buf * 16));
            tc::tmem_wait_ld();
            tc::tc_fence_before();
            tc::mbar_arrive_warp(bar_accfree(buf));
            if (I < nb) {
                const float m = sum / float(min(it.block, a.pool.N - I * it.block));
                const __nv_bfloat16 t1 = __float2bfloat16_rn(m);
                const float r1 = m - __bfloat162float(t1);
                const __nv_bfloat16 t2 = __float2bfloat16_rn(r1);
                const __nv_bfloat16 t3 = __float2bfloat16_rn(r1 - __bfloat162float(t2));
                dst[d] = t1; dst[term_stride + d] = t2; dst[2 * term_stride + d] = t3;
            }
            // A head's counter moves when this CTA leaves the head (one fence per head, not one per block: a fence per
            // batch of two blocks slowed the whole kernel by a fifth).  The named barrier orders the four warps' stores
            // before thread 0's fence.
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
            // Item number -> (head, block): a head's K blocks first, then its Q blocks.  This thread is the pooling path's
            // serial part (a block every 0.7 us at full rate), so an item number is divided only once per batch and
            // stepped from there.
            struct Dec { int base, bh, rem, h, b; };
            auto decode = [&](int item) {
                Dec d; d.base = item; d.bh = item / per_head; d.rem = item - d.bh * per_head; d.b = d.bh / H; d.h = d.bh - d.b * H; return d;
            };
            auto advance = [&](Dec& d) {
                if (++d.rem == per_head) { d.rem = 0; ++d.bh; if (++d.h == H) { d.h = 0; ++d.b; } }
            };
            const int blk_q = a.pool.block[0], blk_k = a.pool.block[1];
            // Items are taken two at a time from the counter (small batches keep the CTAs level and a head's counter
            // moving), but L2 is asked for them 128 KB ahead of the loads: the batches taken and not yet loaded wait,
            // decoded, in a small queue.
            auto prefetch_batch = [&](Dec d) {
                for (int j = 0; j < kBatch && d.base + j < pool_total; ++j, advance(d)) {
                    const int which = d.rem < nki ? 1 : 0;
                    const int row0 = which ? d.rem * PB * blk_k : (d.rem - nki) * PB * blk_q;
                    tma_prefetch_5d(which ? &mapK : &mapQ, 0, row0, 0, d.h, d.b);
                }
            };
            constexpr int kAhead = kFusedAheadBytes / int(L::kSlot) / kBatch;     // batches between counter and load
            static_assert(kAhead >= 1 && kAhead < 8, "look-ahead queue");
            Dec* const ahead = reinterpret_cast<Dec*>(ahead_q);
            for (int k = 0; k < kAhead; ++k) { ahead[k] = decode(atomicAdd(&a.hdr->work[0], kBatch)); prefetch_batch(ahead[k]); }
            int pending = atomicAdd(&a.hdr->work[0], kBatch);       // its value is needed one batch from now: the latency hides
            int armed = -1, n = 0;
            bool more = true;
            for (int nb = 0; more; ++nb) {
                const Dec fresh = decode(pending);
                ahead[(nb + kAhead) & 7] = fresh;
                prefetch_batch(fresh);
                pending = atomicAdd(&a.hdr->work[0], kBatch);
                Dec d = ahead[nb & 7];
                const int base_cur = d.base;
                for (int j = 0; j < kBatch; ++j, ++n, advance(d)) {
                    const int item = base_cur + j;
                    const int s = n % PST;
                    PoolItem it; it.bh = -1; it.I = 0; it.block = 0; it.nvalid = 0;
                    if (n >= PST && !tc::mbar_wait(bar_empty(s), uint32_t(n / PST - 1) & 1u, abortp, 64)) {
                        if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 42, n, blockIdx.x);
                        *abortp = 1; more = false; break;
                    }
                    if (item >= pool_total) {                          // end marker for the MMA warp and the epilogue
                        pool_q[n % kFusedQueue] = it;
                        tc::mbar_arrive(bar_full(s));
                        more = false; break;
                    }
                    const int which = d.rem < nki ? 1 : 0;
                    const int I = (which ? d.rem : d.rem - nki) * PB;      // the item's first block
                    const int block = which ? blk_k : blk_q;
                    it.bh = d.bh; it.I = I | (which << 30); it.block = block;
                    it.nvalid = min(block, a.pool.N - I * block);
                    pool_q[n % kFusedQueue] = it;                      // read by the others only after bar_full / bar_acc of this item
                    tc::mbar_expect_tx(bar_full(s), uint32_t(PB * block) * D * 2);     // rows past N arrive as zeros and count
                    tma_load_5d(smem_base + uint32_t(L::kOffRing + s * L::kSlot), which ? &mapK : &mapQ, bar_full(s),
                                0, I * block, 0, d.h, d.b);               // both halves of the head dimension, or both blocks, in one copy
                    armed = n;
                }
            }
            if (*abortp)       // copies in flight must land before the CTA gives its shared memory back
                for (int k = 0; k < PST && armed - k >= 0; ++k)
                    tc::mbar_wait_drain(bar_full((armed - k) % PST), uint32_t((armed - k) / PST) & 1u);
        }
    } else if (warp_id == 5) {
        // ================= pooling sums on the tensor cores (converged warp, one elected lane issues) =================
        {
            // A = the item, MN-major: rows = head-dimension elements, the second 64 rows one block of 128-byte rows behind
            // the first (D = 128: the second half of the head dimension; D = 64: the next block); B = ones, K-major.
            constexpr uint32_t idesc = tc::instr_desc(128, 16, 0) | (1u << 15);
            const uint64_t db = tc::smem_desc(smem_base + uint32_t(L::kOffOnes), 16, 1024);
            bool ok = true;
            for (int n = 0; ok; ++n) {
                const int s = n % PST, buf = n & 1;
                ok = tc::mbar_wait_warp(bar_full(s), uint32_t(n / PST) & 1u, abortp, 32);
                if (!ok) { if (lane == 0) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 43, n, blockIdx.x); *abortp = 1; } break; }
                const PoolItem it = pool_q[n % kFusedQueue];
                if (n >= 2) {
                    ok = tc::mbar_wait_warp(bar_accfree(buf), uint32_t((n - 2) >> 1) & 1u, abortp, 32);
                    if (!ok) { if (lane == 0) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 44, n, blockIdx.x); *abortp = 1; } break; }
                }
                if (it.bh < 0) { if (lane == 0) tc::mbar_arrive(bar_acc(buf)); break; }              // pass the end marker on
                tc::tc_fence_after();
                const int ksteps = (it.block + 15) / 16;                              // token rows past the valid ones read as zero
                // rows 64-127 of the operand lie one block of 128-byte rows behind rows 0-63
                const uint64_t da = tc::smem_desc(smem_base + uint32_t(L::kOffRing + s * L::kSlot), uint32_t(it.block) * 128u, 1024);
                for (int kk = 0; kk < ksteps; ++kk)
                    mma_ss_elect(tmem + uint32_t(buf * 16), da + uint64_t(kk * (2048 >> 4)), db, idesc, kk > 0 ? 1u : 0u);
                tc::tc_commit_el(bar_acc(buf));
                tc::tc_commit_el(bar_empty(s));
            }
            tc::tc_commit_el(bar_drain);                               // no product may still run when tensor memory is released
            tc::mbar_wait_drain(bar_drain, 0);
            __syncwarp();
        }
    } else if (warp_id == 6) {
        // ================= score producer: the three-term means of an item's query blocks and of the head's key blocks =================
        if (lane == 0) {
            tc::prefetch_tmap(&mapQs); tc::prefetch_tmap(&mapKs);
            const int rows_q = heads * nqb, rows_k = heads * nkb;      // rows of one term in the two mean arrays
            int ready_head = -1, step = 0;                             // A-buffer uses so far
            bool ok = true;
            for (int n = 0; ok; ++n) {
                const int item = atomicAdd(&a.hdr->work[1], 1);
                ScoreItem si; si.bh = -1; si.I0 = 0;
                if (n >= 1) {       // B (and the queue entry two back) is free once the products of the previous item have read it
                    ok = tc::mbar_wait(bar_bfree, uint32_t(n - 1) & 1u, abortp, 64);
                    if (!ok) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 45, n, blockIdx.x); *abortp = 1; break; }
                }
                if (item >= score_total) { score_q[n & 3] = si; tc::mbar_arrive(bar_bfull); break; }
                si.bh = item / groups_per_head;
                si.I0 = (item - si.bh * groups_per_head) * NR;
                if (si.bh != ready_head) {                              // the head's pooled vectors must all be written
                    if (ld_acquire(a.done + si.bh) < per_head) {
                        const unsigned long long t0 = global_timer_ns();
                        ok = false;
                        for (uint32_t it = 0; it < (1u << 30); ++it) {
                            __nanosleep(200);
                            if (ld_acquire(a.done + si.bh) >= per_head) { ok = true; break; }
                            if ((it & 63u) == 63u && (*abortp || global_timer_ns() - t0 > kDefaultWaitNs)) break;
                        }
                        if (!ok) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 40, si.bh, blockIdx.x); *abortp = 1; break; }
                    }
                    ready_head = si.bh;
                    // the means were written with ordinary stores by other SMs; the copies below read them through the async proxy
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                }
                score_q[n & 3] = si;
                tc::mbar_expect_tx(bar_bfull, uint32_t(3 * KH * L::kBoxB));
                for (int t3 = 0; t3 < 3; ++t3)
                    for (int kh = 0; kh < KH; ++kh)
                        tma_load_2d(smem_base + uint32_t(L::kOffScoreB + (t3 * KH + kh) * L::kBoxB), &mapQs, bar_bfull,
                                    kh * 64, t3 * rows_q + si.bh * nqb + si.I0);
                for (int t = 0; t < ntiles && ok; ++t)
                    for (int kq = 0; kq < 2 * KH; ++kq, ++step) {        // quarters of 32 elements, the buffers in turn
                        const int buf = step % AST;
                        if (step >= AST) {
                            ok = tc::mbar_wait(bar_afree(buf), uint32_t(step / AST - 1) & 1u, abortp, 32);
                            if (!ok) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 46, step, blockIdx.x); *abortp = 1; break; }
                        }
                        tc::mbar_expect_tx(bar_afull(buf), uint32_t(3 * L::kBoxA));
                        for (int t3 = 0; t3 < 3; ++t3)
                            tma_load_2d(smem_base + uint32_t(L::kOffScoreA + (buf * 3 + t3) * L::kBoxA), &mapKs, bar_afull(buf),
                                        kq * 32, t3 * rows_k + si.bh * nkb + t * 128);
                    }
            }
            // on the way out after an abort, copies in flight must land first; an unarmed barrier simply runs out
            if (*abortp)
                for (int k = 1; k <= AST && step - k >= 0; ++k)
                    tc::mbar_wait_drain(bar_afull((step - k) % AST), uint32_t((step - k) / AST) & 1u, 20000000ull);
        }
    } else if (warp_id == 7) {
        // ================= scores on the tensor cores (converged warp, one elected lane issues) =================
        {
            // S^T tile t (128 key blocks x 16 query blocks) += A_term x B_term^T over the six term pairs, 16 elements of
            // the head dimension per instruction; both operands K-major (rows of 128 B, 128-byte swizzle).
            constexpr uint32_t idesc = tc::instr_desc(128, NR, 0);
            const uint64_t da0 = tc::smem_desc_sw64(smem_base + uint32_t(L::kOffScoreA), 16, 512);
            const uint64_t db0 = tc::smem_desc(smem_base + uint32_t(L::kOffScoreB), 16, 1024);
            constexpr int pa[6] = {0, 0, 1, 0, 1, 2}, pb[6] = {0, 1, 0, 2, 1, 0};       // term pairs, largest products first
            int step = 0;
            bool ok = true;
            for (int n = 0; ok; ++n) {
                ok = tc::mbar_wait_warp(bar_bfull, uint32_t(n) & 1u, abortp, 32);
                if (!ok) { if (lane == 0) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 47, n, blockIdx.x); *abortp = 1; } break; }
                const ScoreItem si = score_q[n & 3];
                if (n >= 1) {       // the selection group has moved the previous item's scores out of tensor memory
                    ok = tc::mbar_wait_warp(bar_sfree, uint32_t(n - 1) & 1u, abortp, 32);
                    if (!ok) { if (lane == 0) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 48, n, blockIdx.x); *abortp = 1; } break; }
                }
                if (si.bh < 0) { if (lane == 0) tc::mbar_arrive(bar_sfull); break; }                   // pass the end marker on
                for (int t = 0; t < ntiles && ok; ++t)
                    for (int kq = 0; kq < 2 * KH; ++kq, ++step) {
                        const int buf = step % AST, kh = kq >> 1;
                        ok = tc::mbar_wait_warp(bar_afull(buf), uint32_t(step / AST) & 1u, abortp, 32);
                        if (!ok) { if (lane == 0) { if (!*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 49, step, blockIdx.x); *abortp = 1; } break; }
                        tc::tc_fence_after();
                        // The tensor cores add into an fp32 accumulator without guard bits, so a long chain of additions
                        // at the magnitude of the score loses a few bits.  The leading product t1 t1 (the only large one)
                        // therefore has an accumulator per half of the head dimension (four additions each); the five
                        // small products share another.  The selection group adds them in fp32.
                        const uint32_t d_tile = tmem_s + uint32_t(t * NR * NACC);
                        const uint32_t d_big = d_tile + uint32_t((NACC == 2 ? 0 : kh) * NR), d_small = d_tile + uint32_t((NACC - 1) * NR);
                        const bool big_first = NACC == 2 ? kq == 0 : (kq & 1) == 0;
#pragma unroll
                        for (int p = 0; p < 6; ++p)
#pragma unroll
                            for (int kk = 0; kk < 2; ++kk)
                                mma_ss_elect(p == 0 ? d_big : d_small,
                                           da0 + uint64_t(((buf * 3 + pa[p]) * L::kBoxA + kk * 32) >> 4),
                                           db0 + uint64_t(((pb[p] * KH + kh) * L::kBoxB + (kq & 1) * 64 + kk * 32) >> 4),
                                           idesc, p == 0 ? ((!big_first || kk > 0) ? 1u : 0u) : ((kq > 0 || p > 1 || kk > 0) ? 1u : 0u));
                        tc::tc_commit_el(bar_afree(buf));
                    }
                if (!ok) break;
                tc::tc_commit_el(bar_bfree);
                tc::tc_commit_el(bar_sfull);
            }
            tc::tc_commit_el(bar_drain2);
            tc::mbar_wait_drain(bar_drain2, 0);
            __syncwarp();
        }
    } else {
    // ================= selection group =================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 96;" ::: "memory");
    const int t = tid - kFusedPoolThreads;
    constexpr int NT = kFusedScoreThreads;
    constexpr int NW = NT / 32;                                        // 16 warps = kFusedRows: one query block per warp
    static_assert(NW == kFusedRows, "one selection warp per row of an item");
    float* sS = reinterpret_cast<float*>(fsm + L::off_scores(nkb));  // [RP][nkb_pad]
    const Geometry g = a.sel.g;
    const int warp = t >> 5;
    const int quarter = warp & 3;                                      // tensor-memory lanes this warp may read
    const uint32_t lane_base = uint32_t(quarter * 32) << 16;
    const int text_cols = (g.text_dense && g.n_text > 0) ? (g.n_text + g.bk - 1) / g.bk : 0;
    bool ok = true;
    for (int n = 0; ok; ++n) {
        ok = tc::mbar_wait_warp(bar_sfull, uint32_t(n) & 1u, abortp, 64);
        if (!ok) { if (lane == 0 && !*abortp) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 50, n, blockIdx.x); break; }
        const ScoreItem si = score_q[n & 3];
        if (si.bh < 0) break;
        const int bh = si.bh, I0 = si.I0;
        const int nrows = min(NR, nqb - I0);
        tc::tc_fence_after();
        constexpr int TPW = 2;                                         // score tiles a warp reads at most (8 tiles, 4 warps per lane quarter)
        float v[TPW][16];                                              // with 8-row passes an even pass reads for the odd one after it as well
        constexpr int kLastRead = RP == 16 ? NR / RP - 1 : NR / RP - 2;
#pragma unroll 1
        for (int pass = 0; pass < NR / RP; ++pass) {
        // ---- tensor memory -> registers: a thread holds one key block's scores against 16 of the item's query blocks ----
        const int c0 = ((pass * RP) / 16) * 16;                        // first of the 16 accumulator columns read in this pass
        if (RP == 16 || (pass & 1) == 0) {
#pragma unroll
            for (int j = 0; j < TPW; ++j) {
                const int tile = (warp >> 2) + j * (NW / 4);
                if (tile < ntiles) {                                   // warp-uniform
                    float u[16];
                    tmem_ld16(tmem_s + lane_base + uint32_t(tile * NR * NACC + c0), v[j]);                        // t1 t1 (first half of d)
                    tmem_ld16(tmem_s + lane_base + uint32_t(tile * NR * NACC + (NACC - 1) * NR + c0), u);         // the small products
                    tc::tmem_wait_ld();
                    if (NACC == 3) {
                        float v2[16];
                        tmem_ld16(tmem_s + lane_base + uint32_t(tile * NR * NACC + NR + c0), v2);                  // t1 t1, second half
                        tc::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[j][i] += v2[i];
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[j][i] = a.scale * (v[j][i] + u[i]);
                }
            }
        }
        if (pass == kLastRead) {       // the last columns are in registers: the next item's products may overwrite the tiles
            tc::tc_fence_before();
            tc::mbar_arrive_warp(bar_sfree);
        }
        // ---- RP rows into shared memory (one row per query block), then one warp per row selects ----
#pragma unroll
        for (int j = 0; j < TPW; ++j) {
            const int tile = (warp >> 2) + j * (NW / 4);
            const int J = tile * 128 + quarter * 32 + lane;
            if (tile < ntiles && J < nkb) {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (RP == 16 || i / 8 == (pass & 1)) sS[(i % RP) * a.nkb_pad + J] = v[j][i];
            }
        }
        named_bar(2, NT);
        const int rsel = pass * RP + warp;                              // row of the item this warp selects for
        if (warp < RP && rsel < nrows) {
            const int I = I0 + rsel;
            const float* srow = sS + warp * a.nkb_pad;
            const int64_t row = (int64_t(bh) * nqb + I) * nkb;
            const bool text_row = g.text_dense && g.n_text > 0 && I * g.bq < g.n_text;
            // Always-kept key blocks of the frame window: blocks are runs of consecutive tokens, so the blocks that touch
            // frames [f_lo, f_hi] are the interval [j_lo, j_hi] of blocks that touch tokens [n_text + f_lo hw, n_text + (f_hi + 1) hw).
            int j_lo = 1, j_hi = 0;
            if (g.window >= 0) {
                const int q_lo = max(I * g.bq, g.n_text), q_hi = min(g.N, (I + 1) * g.bq) - 1;
                if (q_hi >= q_lo) {
                    const int f_lo = max(0, (q_lo - g.n_text) / g.hw - g.window);
                    const int f_hi = min(g.T - 1, (q_hi - g.n_text) / g.hw + g.window);
                    j_lo = (g.n_text + f_lo * g.hw) / g.bk;
                    j_hi = (min(g.N, g.n_text + (f_hi + 1) * g.hw) - 1) / g.bk;
                }
            }
            if (text_row) { j_lo = 0; j_hi = nkb - 1; }
            uint32_t key[NPL];
            uint32_t forced_bits[(NPL + 31) / 32];
#pragma unroll
            for (int w = 0; w < (NPL + 31) / 32; ++w) forced_bits[w] = 0u;
            int my_forced = 0;
#pragma unroll
            for (int q = 0; q < NPL; ++q) {
                const int J = q * 32 + lane;
                uint32_t k = 0u;                                        // always-kept and out-of-range entries never compete
                if (J < nkb) {
                    const float sv = srow[J];
                    const bool forced = J < text_cols || (J >= j_lo && J <= j_hi);
                    if (forced) { forced_bits[q >> 5] |= 1u << (q & 31); ++my_forced; }
                    else k = ordered_bits(sv);
                    if (a.scores_out) a.scores_out[row + J] = sv;
                }
                key[q] = k;
            }
            const int nforced = __reduce_add_sync(0xffffffffu, my_forced);
            const int nfree = nkb - nforced;
            int n_admit = a.sel.count_includes_forced ? max(0, a.sel.k_all - nforced) : topk_count_dev(a.sel.keep_ratio, nfree);
            n_admit = min(n_admit, nfree);
            // k-th largest key, bit by bit: the largest T with #(key >= T) >= n_admit.  Once a candidate is met by exactly
            // n_admit keys the kept set is known (the remaining bits would only find its smallest key).
            // Bits above the first one in which two competing keys differ are the same in T as in every such key: they
            // are taken over at once (keys of always-kept and absent blocks are 0 and never compete).
            uint32_t k_or = 0u, k_and = 0xFFFFFFFFu;
#pragma unroll
            for (int q = 0; q < NPL; ++q) { k_or |= key[q]; k_and &= key[q] ? key[q] : 0xFFFFFFFFu; }
            k_or = __reduce_or_sync(0xffffffffu, k_or);
            k_and = __reduce_and_sync(0xffffffffu, k_and);
            const int top = 31 - __clz(int((k_or ^ k_and) | 1u));       // highest bit in which competing keys differ (0 if none do)
            uint32_t T = (top >= 31) ? 0u : (k_and & ~((2u << top) - 1u));
            bool exact = n_admit == 0;
#pragma unroll 1
            for (int bit = top; bit >= 0 && !exact; --bit) {
                const uint32_t cand = T | (1u << bit);
                int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
                for (int q = 0; q + 3 < NPL; q += 4) {
                    c0 += (key[q] >= cand) ? 1 : 0; c1 += (key[q + 1] >= cand) ? 1 : 0;
                    c2 += (key[q + 2] >= cand) ? 1 : 0; c3 += (key[q + 3] >= cand) ? 1 : 0;
                }
                const int c = __reduce_add_sync(0xffffffffu, (c0 + c1) + (c2 + c3));
                if (c >= n_admit) { T = cand; exact = (c == n_admit); }
            }
            const bool any = n_admit > 0;                               // n_admit == 0: nothing is admitted by score
            if (exact) {
                // The search ended on a threshold that exactly n_admit keys reach (or nothing is admitted): every key
                // at or above it is kept and no tie has to be broken.  Keys of always-kept and absent blocks are 0 < T.
#pragma unroll
                for (int q = 0; q < NPL; ++q) {
                    const int J = q * 32 + lane;
                    const bool keep = ((forced_bits[q >> 5] >> (q & 31)) & 1u) || (any && key[q] >= T);
                    if (J < nkb) a.sel.mask[row + J] = keep ? 1 : 0;
                }
            } else {
                int gt = 0;
#pragma unroll
                for (int q = 0; q < NPL; ++q) gt += (key[q] > T) ? 1 : 0;
                gt = __reduce_add_sync(0xffffffffu, gt);
                const int need_eq = n_admit - gt;                       // blocks with key == T, lowest block index first
                int seen_eq = 0;
#pragma unroll
                for (int q = 0; q < NPL; ++q) {
                    const int J = q * 32 + lane;
                    const bool eq = key[q] == T;
                    const unsigned bal = __ballot_sync(0xffffffffu, eq);
                    const int rank = seen_eq + __popc(bal & ((1u << lane) - 1u));
                    seen_eq += __popc(bal);
                    const bool keep = ((forced_bits[q >> 5] >> (q & 31)) & 1u) || key[q] > T || (eq && rank < need_eq);
                    if (J < nkb) a.sel.mask[row + J] = keep ? 1 : 0;
                }
            }
        }
        named_bar(2, NT);                                              // the rows are free for the next pass / item
        }
    }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp_id == 5) {
        tc::tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kFusedTmemCols) : "memory");
    }
}

}  // namespace carnator
