// Block-sparse attention on the 5th-generation tensor cores: TMA loads of the listed K/V tiles,
// tcgen05.mma with S = Q K^T and O += P V accumulated in tensor memory, online softmax in the
// consumer warps.  One CTA per (batch, head, query block) of 128 queries; key blocks of 128.
// Paper: Section 3.3, "Historical Sparse-Connectivity Reuse" (only the block pairs the historical
// structure lists are evaluated; Q, K, V are the target's own).
//
// Warp roles (384 threads = three warpgroups, one CTA per SM):
//   warps 0-3  softmax group 0, warps 4-7 softmax group 1: the groups take the 128-key steps in turn; within
//              a group warp w owns tensor-memory lanes 32w..32w+31 = query rows.  Both also run the epilogue.
//   warp 8     TMA producer for the K tiles (one lane)
//   warp 9     tensor-memory allocation, issue of every matrix product (the warp stays converged, an elected lane issues)
//   warp 10    TMA producer for the V tiles (one lane)
//   warp 11    idle
// The third warpgroup gives most of its registers to the softmax groups (setmaxnreg), which hold a full
// 128-column score row per thread.
// One warp issues all the matrix products: two threads issuing at once each ran at half the rate, and the
// pipe then executes in a known order.  The warp runs its loop converged and elects the issuing lane per instruction
// (elect.sync) instead of sending one lane into a branch: the descriptors then live in uniform registers and a batch
// takes a third fewer cycles to queue while the softmax warps on the same scheduler are busy.  Each batch ends in
// one tcgen05.commit (a commit costs the issuer about as much as two MMAs): "S_g full" also releases the K slot,
// "P V done" also releases the V slot and the P buffer.
// Tensor memory (512 columns): S0 | S1 (128 fp32 columns each, one per softmax group), P (64 columns of packed
// bf16), Q (D / 2 columns of packed bf16), O (D fp32 columns).  The query tile is written there once by the
// softmax groups (straight from global memory) and serves as the A operand of every Q K^T, so those products
// read only the K tile from shared memory, whose bandwidth the TMA writes and the operand reads share.  A group
// signals as soon as it has pulled its scores into registers, so Q K^T of its next step runs underneath its own
// exponentials; it keeps its probabilities in registers until they are complete and stores them in one go, by
// which time P V of the previous step has long read the one P buffer.  P V is issued in step order.
// Every wait on an mbarrier is bounded; on expiry the role records CARNATOR_ERR_DEVICE_TIMEOUT in
// the workspace header, raises a CTA-wide abort flag, and every role drains and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "attn_portable.cuh"

namespace carnator {
namespace tc {

constexpr int kBlock = 128;            // query rows per CTA = keys per step
constexpr int kSBufs = 2;              // score buffers in tensor memory, one per softmax group
constexpr int kRefSlots = 3;           // hand-over slots of the shared reference maximum
constexpr int kStages = 3;             // ring slots for K tiles and for V tiles
constexpr int kSoftmaxWarps = 8;       // two warpgroups taking the steps in turn
constexpr int kThreads = (kSoftmaxWarps + 4) * 32;   // third warpgroup: two TMA producers, the MMA issuer, one idle warp
constexpr int kWarpTmaK = 8, kWarpMma = 9, kWarpTmaV = 10;
constexpr int kTmemCols = 512;         // S0 | S1 | P | Q | O
constexpr uint32_t kColP = 2 * kBlock;        // packed bf16 probabilities: 64 columns, one buffer for both groups
constexpr uint32_t kColQ = 2 * kBlock + 64;   // the query tile as packed bf16 pairs: D / 2 columns (A operand of Q K^T)
constexpr uint32_t kColO = 2 * kBlock + 2 * 64;
constexpr int kRegsService = 72, kRegsSoftmax = 216;   // setmaxnreg targets (the literals in the kernel must match)
constexpr float kRescaleThreshold = 8.0f;   // log2 units: P stays below 2^8, well inside bf16/fp32 range

// ---- small PTX wrappers -----------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done;
}
// Non-blocking form for polling loops: try_wait may suspend the thread for a while when the phase is not complete.
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after limit_ns (or when another role has aborted) and raises the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned sleep_ns = 0,
                                          unsigned long long limit_ns = kDefaultWaitNs) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0; it < (1u << 30); ++it) {
        if (sleep_ns) __nanosleep(sleep_ns);
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 255u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    return false;
}

// Wait used on the way out, after an abort: the copies or products this role still has in flight must land before
// the CTA gives its shared and tensor memory back, so the abort flag does not end this wait; only time does.
__device__ __forceinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity, unsigned long long limit_ns = kDefaultWaitNs) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0; it < (1u << 30); ++it) {
        __nanosleep(100);
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 255u && global_ns() - t0 > limit_ns) break;
    }
    return false;
}

// Warp-collective form.  Every lane tests the barrier (one broadcast read of shared memory, no divergence in the
// common case that the phase is already complete); lanes that find it incomplete fall into the bounded wait.  The
// vote makes the outcome uniform, reconverges the warp and orders the other lanes' later reads after the acquire.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned sleep_ns = 0,
                                               unsigned long long limit_ns = kDefaultWaitNs) {
    const bool ok = mbar_try(bar, parity) ? true : mbar_wait(bar, parity, abort_flag, sleep_ns, limit_ns);
    return __all_sync(0xffffffffu, ok) != 0;
}
// One arrival per warp once every lane's earlier writes are ordered before it.
__device__ __forceinline__ void mbar_arrive_warp(uint32_t bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Same with the descriptors given as (low word, shared high word): the issuing thread keeps the low words in
// registers and only adds a constant per instruction, which keeps its dependent instruction chain short.
__device__ __forceinline__ void mma_ss_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_ts_lo(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// Forms for a converged warp: every lane executes the statement with the same operands and one elected lane issues
// the instruction.  The compiler can then keep the descriptors in uniform registers, and queuing a batch costs the
// warp far fewer issue slots than it does from inside a one-lane branch: measured with two softmax groups running on
// the same SM, 54 clk per instruction against 79.
__device__ __forceinline__ void mma_ts_el(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "elect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_el(uint32_t bar) {
    asm volatile(
        "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}
// Two fp32 lanes per instruction (packed pair in a 64-bit register): halves the FMA-pipe instruction count of the
// exponent arguments and of the row sums.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// ---- descriptors --------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1 (bit 46), layout type 2 = SWIZZLE_128B (bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return uint64_t((addr & 0x3FFFFu) >> 4)
         | (uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16)
         | (uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32)
         | (1ull << 46)
         | (2ull << 61);
}
// Same with the 64-byte swizzle (rows of 64 B, atoms of 8 rows = 512 B): layout type 4.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return uint64_t((addr & 0x3FFFFu) >> 4)
         | (uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16)
         | (uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32)
         | (1ull << 46)
         | (4ull << 61);
}
// Instruction descriptor for kind::f16: fp32 accumulator, bf16 x bf16, M x N, B operand major-ness.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(b_mn_major) << 16) | (uint32_t(N >> 3) << 17) | (uint32_t(M >> 4) << 24);
}

// Shared-memory plan.  Every K / V tile is 128 rows x D held as D/64 boxes of 128 rows x 128 B
// (128-byte swizzle).  K and V tiles travel through kStages-slot rings (separate rings, separate producers).
template <int D>
struct Cfg {
    static constexpr int kBoxes = D / 64;
    static constexpr uint32_t kBoxBytes = kBlock * 128;             // 128 rows x 128 B
    static constexpr uint32_t kTileBytes = kBoxes * kBoxBytes;      // one 128 x D bf16 tile
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffV = kOffK + kStages * kTileBytes;
    static constexpr uint32_t kOffBar = kOffV + kStages * kTileBytes;
    static constexpr uint32_t kSmemBytes = kOffBar + 512 + 1024;    // barriers + slack to align the base to 1 KiB
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, const AttnArgs a) {
    using C = Cfg<D>;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float r_pub[kRefSlots][kBlock];     // reference maximum after step i, slot i % 3 (handed from one warpgroup to the other)
    __shared__ float fin[2][2][kBlock];         // per warpgroup: final reference maximum and partial row sum

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.z, h = blockIdx.y;
    const int64_t bh = int64_t(b) * a.H + h;
    const int I = a.order[bh * a.nqb + blockIdx.x];
    const int T = a.counts[bh * a.nqb + I];           // steps = listed key blocks
    const int32_t* list = a.lists + (bh * a.nqb + I) * int64_t(a.nkb);
    const int q0 = I * kBlock;

    if (T < 0) return;                      // skipped query block (region-restricted form): output untouched
    if (T > a.nkb) {                        // a count that cannot come from compaction: stop before reading a list that long
        if (tid == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_CHECK, 20, T, blockIdx.x);
        return;
    }
    if (T == 0) {                           // nothing to attend to: O = 0, LSE = -inf
        if (tid < kBlock && q0 + tid < a.N) {
            __nv_bfloat16* op = a.O + b * a.os[0] + h * a.os[1] + int64_t(q0 + tid) * a.os[2];
#pragma unroll
            for (int c = 0; c < D / 8; ++c) *reinterpret_cast<uint4*>(op + c * 8) = make_uint4(0, 0, 0, 0);
            a.LSE[bh * a.N + q0 + tid] = -INFINITY;
        }
        return;
    }

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t sK = smem_base + C::kOffK;
    const uint32_t sV = smem_base + C::kOffV;
    const uint32_t bars = smem_base + C::kOffBar;
    const uint32_t bar_q = bars, bar_o = bars + 8, bar_drain = bars + 16;
    auto bar_kfull = [&](int s) { return bars + 32 + 8 * s; };       // up to 4 stages each
    auto bar_vfull = [&](int s) { return bars + 96 + 8 * s; };
    auto bar_sfull = [&](int s) { return bars + 160 + 8 * s; };      // S_g holds fresh scores
    auto bar_sfree = [&](int s) { return bars + 176 + 8 * s; };      // group g has read S_g into registers
    auto bar_pfull = [&](int s) { return bars + 192 + 8 * s; };      // P_g is complete
    auto bar_ref = [&](int s, int q) { return bars + 224 + 8 * (s * 4 + q); };   // r_pub slot s, lane quarter q
    auto bar_fin = [&](int q) { return bars + 320 + 8 * q; };
    auto bar_pvdone = [&](int s) { return bars + 352 + 8 * s; };     // P V of the step that used score buffer s has completed
    volatile int* abortp = &abort_flag;
    // every bounded wait of this CTA gives up after `limit` (2 s unless the workspace header asks for less)
    const unsigned long long limit = a.hdr->wait_limit_ns ? a.hdr->wait_limit_ns : kDefaultWaitNs;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_q, kSoftmaxWarps); mbar_init(bar_o, 1); mbar_init(bar_drain, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_kfull(s), 1); mbar_init(bar_vfull(s), 1);
        }
        for (int s = 0; s < kSBufs; ++s) {
            mbar_init(bar_sfull(s), 1); mbar_init(bar_pvdone(s), 1);
            mbar_init(bar_pfull(s), 4); mbar_init(bar_sfree(s), 4);          // one arrival per softmax warp of the group
        }
        for (int s = 0; s < kRefSlots; ++s)
            for (int q = 0; q < 4; ++q) mbar_init(bar_ref(s, q), 1);
        for (int q = 0; q < 4; ++q) mbar_init(bar_fin(q), 2);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kWarpTmaK && lane == 0) prefetch_tmap(&mapK);
    if (warp == kWarpTmaV && lane == 0) prefetch_tmap(&mapV);
    if (warp == kWarpMma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    if (warp >= kSoftmaxWarps) {
    // Register budget: the producer / MMA warpgroup needs few registers and hands the rest to the softmax groups.
    // The CTA is launched with 384 x 168 registers; 256 x 216 + 128 x 72 uses exactly that.  A split that asks for
    // more makes setmaxnreg.inc wait for registers that never come.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;" ::: "memory");
    if (warp == kWarpTmaK) {
        // ================= TMA producer: the K tiles =================
        if (lane == 0) {
            int armed = -1;
            for (int i = 0; i < T; ++i) {
                const int s = i % kStages, u = i - kStages;     // the slot is free once Q K^T of step u has completed
                if (u >= 0 && !mbar_wait(bar_sfull(u & 1), uint32_t(u >> 1) & 1u, abortp, 100, limit)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 1, i, blockIdx.x); break;
                }
                const int J = list[i];
                if (J < 0 || J >= a.nkb || (i > 0 && J <= list[i - 1])) {      // malformed list: stop before touching memory
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_CHECK, 21, i, blockIdx.x); *abortp = 1; break;
                }
                // Test of the time-out path only: the first K tile of the first query block in the order is never
                // requested, so the wait for it runs out and the CTA takes the abort-and-drain path.
                if (i == 0 && a.hdr->debug_withhold != 0 && blockIdx.x == 0 && bh == 0) continue;
                mbar_expect_tx(bar_kfull(s), C::kTileBytes);
                const int key0 = J * kBlock;
#pragma unroll
                for (int x = 0; x < C::kBoxes; ++x)
                    tma_load_4d(sK + s * C::kTileBytes + x * C::kBoxBytes, &mapK, bar_kfull(s), x * 64, key0, h, b);
                armed = i;
            }
            if (*abortp) {      // copies in flight must land before the CTA gives its shared memory back
                for (int k = 0; k < kStages && armed - k >= 0; ++k)
                    mbar_wait_drain(bar_kfull((armed - k) % kStages), uint32_t((armed - k) / kStages) & 1u, limit);
            }
        }
    } else if (warp == kWarpTmaV) {
        // ================= TMA producer: the V tiles =================
        if (lane == 0) {
            int armed = -1;
            for (int i = 0; i < T; ++i) {
                const int s = i % kStages, u = i - kStages;     // the slot is free once P V of step u has completed
                if (u >= 0 && !mbar_wait(bar_pvdone(u & 1), uint32_t(u >> 1) & 1u, abortp, 100, limit)) {
                    set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 2, i, blockIdx.x); break;
                }
                const int J = list[i];
                if (J < 0 || J >= a.nkb) { *abortp = 1; break; }                  // reported by the K producer
                mbar_expect_tx(bar_vfull(s), C::kTileBytes);
                const int key0 = J * kBlock;
#pragma unroll
                for (int x = 0; x < C::kBoxes; ++x)
                    tma_load_4d(sV + s * C::kTileBytes + x * C::kBoxBytes, &mapV, bar_vfull(s), x * 64, key0, h, b);
                armed = i;
            }
            if (*abortp) {
                for (int k = 0; k < kStages && armed - k >= 0; ++k)
                    mbar_wait_drain(bar_vfull((armed - k) % kStages), uint32_t((armed - k) / kStages) & 1u, limit);
            }
        }
    } else if (warp == kWarpMma) {
        // ================= MMA issuer =================
        // One thread queues every matrix product and serves whichever is ready: Q K^T of the next step (its K tile
        // has landed and the softmax group has taken the previous scores out of that S buffer) or P V of the oldest
        // step whose probabilities are complete.  One commit per batch: the barrier that says "S_g is full" also
        // frees the K slot, and the one that says "P V done" also frees the V slot and P_g.
        // The whole warp runs this loop converged (every decision is a warp vote), and one elected lane issues.
        {
            constexpr uint32_t idesc_qk = instr_desc(kBlock, kBlock, 0);
            constexpr uint32_t idesc_pv = instr_desc(kBlock, D, 1);
            // descriptor words that do not change: low word = (address >> 4) | leading offset; high word = stride
            // offset | version | swizzle mode (see smem_desc)
            const uint64_t dk = smem_desc(sK, 16, 1024), dv = smem_desc(sV, C::kBoxBytes, 1024);
            const uint32_t k_lo0 = uint32_t(dk), hi_kmajor = uint32_t(dk >> 32);
            const uint32_t v_lo0 = uint32_t(dv), hi_v = uint32_t(dv >> 32);
            bool ok = mbar_wait_warp(bar_q, 0, abortp, 0, limit);   // the softmax groups have put the query tile into tensor memory
            if (!ok && lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 3, 0, blockIdx.x);
            tc_fence_after();
            int iq = 0, ip = 0;                          // next Q K^T step, next P V step
            unsigned long long t_idle = 0;               // lane 0's clock decides about giving up
            uint32_t idle = 0;
            while (ip < T && ok) {
                bool progress = false;
                if (ip < iq) {
                    const int s = ip % kStages, g = ip & 1;
                    const bool ready = mbar_test(bar_pfull(g), uint32_t(ip >> 1) & 1u) && mbar_test(bar_vfull(s), uint32_t(ip / kStages) & 1u);
                    if (__all_sync(0xffffffffu, ready)) {
                        // O += P_i V_i : P from tensor memory (16 keys = 8 packed columns per instruction), V tile as the
                        // MN-major B operand (rows = keys, 64-element chunks of the head dimension one box apart)
                        tc_fence_after();
                        const uint32_t v_lo = v_lo0 + uint32_t(s) * (C::kTileBytes >> 4), p_t = tmem + kColP, d_o = tmem + kColO;
                        const uint32_t acc0 = ip > 0 ? 1u : 0u;
#pragma unroll
                        for (int kk = 0; kk < kBlock / 16; ++kk)
                            mma_ts_el(d_o, p_t + kk * 8, v_lo + kk * (2048 >> 4), hi_v, idesc_pv, kk > 0 ? 1u : acc0);
                        tc_commit_el(bar_pvdone(g));
                        ++ip; progress = true;
                    }
                }
                if (iq < T) {
                    const int s = iq % kStages, g = iq & 1;
                    const bool ready = mbar_test(bar_kfull(s), uint32_t(iq / kStages) & 1u) &&
                                       (iq < 2 || mbar_test(bar_sfree(g), uint32_t((iq - 2) >> 1) & 1u));
                    if (__all_sync(0xffffffffu, ready)) {
                        // S_g = Q K_i^T: Q from tensor memory, K tile K-major, 16 elements of the head dimension per instruction
                        tc_fence_after();
                        const uint32_t k_lo = k_lo0 + uint32_t(s) * (C::kTileBytes >> 4), d_s = tmem + g * kBlock;
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off16 = ((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4;      // compile-time constant
                            mma_ts_el(d_s, tmem + kColQ + kk * 8, k_lo + off16, hi_kmajor, idesc_qk, kk > 0 ? 1u : 0u);
                        }
                        tc_commit_el(bar_sfull(g));
                        ++iq; progress = true;
                    }
                }
                if (progress) { idle = 0; continue; }
                __nanosleep(20);                        // keep the polling from taking issue slots from the softmax warps on this scheduler
                if ((++idle & 1023u) == 0) {             // nothing was ready: bounded, like every other wait
                    int give_up = 0;
                    if (lane == 0) {
                        if (*abortp) give_up = 1;
                        else {
                            const unsigned long long now = global_ns();
                            if (idle == 1024u) t_idle = now;
                            else if (now - t_idle > limit) give_up = 2;
                        }
                    }
                    give_up = __shfl_sync(0xffffffffu, give_up, 0);
                    if (give_up) {
                        if (give_up == 2 && lane == 0) { set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 4, ip, blockIdx.x); *abortp = 1; }
                        ok = false;
                        break;
                    }
                }
            }
            if (ok) tc_commit_el(bar_o);
            if (__any_sync(0xffffffffu, *abortp != 0)) {      // make sure no MMA of this warp is still running before tensor memory is released
                tc_commit_el(bar_drain);
                mbar_wait_drain(bar_drain, 0, limit);
                __syncwarp();
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;" ::: "memory");
        // ================= softmax + epilogue (warps 0-7) =================
        // Two warpgroups take the steps in turn (group g: steps g, g+2, ...), each with one warp per
        // tensor-memory lane quarter, so one group's exponentials run while the other group's scores are
        // being produced.  Both feed the same O accumulator, so they share one reference maximum per row:
        // the group that handles step i derives R_i from R_{i-1} (published by the other group right after
        // its row-maximum pass) and publishes R_i in turn.  The reference only moves when a row maximum
        // exceeds it by more than the threshold; then this group rescales O before delivering P_i.
        const int quarter = warp & 3, wg = warp >> 2;
        const int r_loc = quarter * 32 + lane;                      // query row within the tile
        const uint32_t lane_base = uint32_t(quarter * 32) << 16;
        const int row = q0 + r_loc;
        {
            // The query tile goes into tensor memory as the A operand of Q K^T (row = lane, two bf16 per column), so
            // those products read only the K tile from shared memory.  Group g brings half of the head dimension.
            const __nv_bfloat16* qp = a.Q + b * a.qs[0] + h * a.qs[1] + int64_t(row) * a.qs[2] + wg * (D / 2);
#pragma unroll
            for (int c = 0; c < D / 128; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint4 u = row < a.N ? *reinterpret_cast<const uint4*>(qp + c * 64 + v * 8) : make_uint4(0, 0, 0, 0);
                    r[4 * v] = u.x; r[4 * v + 1] = u.y; r[4 * v + 2] = u.z; r[4 * v + 3] = u.w;
                }
                tmem_st32(tmem + lane_base + kColQ + wg * (D / 4) + c * 32, r);
            }
            if (D == 64) {
                uint32_t r[16];
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint4 u = row < a.N ? *reinterpret_cast<const uint4*>(qp + v * 8) : make_uint4(0, 0, 0, 0);
                    r[4 * v] = u.x; r[4 * v + 1] = u.y; r[4 * v + 2] = u.z; r[4 * v + 3] = u.w;
                }
                tmem_st16(tmem + lane_base + kColQ + wg * 16, r);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive_warp(bar_q);
        }
        float m_w = -INFINITY, l_w = 0.f;                           // this group's reference and partial row sum
        bool ok = true;
        // lists ascend, so only the last listed block can be the ragged one: read it once, off the per-step path
        const int nvalid_last = a.N - list[T - 1] * kBlock;
        for (int i = wg; i < T; i += 2) {
            const int rs = i % kRefSlots;
            const uint32_t sph = uint32_t(i >> 1) & 1u;
            ok = mbar_wait_warp(bar_sfull(wg), sph, abortp, 20, limit);   // warp-uniform: the loads below are collective
            if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 7, i, blockIdx.x); break; }
            tc_fence_after();
            const int nvalid = (i == T - 1) ? nvalid_last : kBlock;      // >= 1; < 128 only for a ragged last block
            const uint32_t tS = tmem + lane_base + wg * kBlock;
            const uint32_t tP = tmem + lane_base + kColP;
            float s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s[c]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive_warp(bar_sfree(wg));     // the scores are in registers: S_g may take the scores of step i+2
            if (nvalid < kBlock) {               // ragged tail (warp-uniform): keys >= N never count
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e >= nvalid) s[c][e] = -INFINITY;
            }
            // row maximum of the raw scores (the scale is positive), four independent chains
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 2) mx4[(e >> 1) & 3] = max3(mx4[(e >> 1) & 3], s[c][e], s[c][e + 1]);
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
            // reference handed over from step i-1
            float r_prev = -INFINITY, r_now = mx;
            bool grow = false;
            if (i > 0) {
                ok = mbar_wait_warp(bar_ref((i - 1) % kRefSlots, quarter), uint32_t((i - 1) / kRefSlots) & 1u, abortp, 0, limit);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 10, i, blockIdx.x); break; }
                r_prev = r_pub[(i - 1) % kRefSlots][r_loc];
                grow = mx > r_prev + kRescaleThreshold;
                r_now = grow ? mx : r_prev;
            }
            r_pub[rs][r_loc] = r_now;
            mbar_arrive_warp(bar_ref(rs, quarter));
            // The one P buffer is free again once P V of step i-1 (the other group's) has read it.  The probabilities
            // are kept in registers until they are all there, so that wait comes after the exponentials; the rescaling
            // path needs the same product to be complete (O quiescent) and takes the wait early.  Each step waits on
            // the phase that follows the one it waited on two steps earlier, so the phase is never ambiguous.
            bool p_free = i < 1;
            if (i > 0 && __any_sync(0xffffffffu, grow)) {
                p_free = true;
                // O must be quiescent: P V of step i-1 (the other group's) complete.  P V is issued in step order
                // and that of step i cannot start before this group delivers P_i.
                ok = mbar_wait_warp(bar_pvdone(wg ^ 1), uint32_t((i - 1) >> 1) & 1u, abortp, 0, limit);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 9, i, blockIdx.x); break; }
                tc_fence_after();
                const float f = ex2_approx(r_prev - r_now);          // 1 for rows that did not move
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    float o[32];
                    tmem_ld32(tmem + lane_base + kColO + c * 32, o);
                    tmem_wait_ld();
                    uint32_t r[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(o[e] * f);
                    tmem_st32(tmem + lane_base + kColO + c * 32, r);
                }
            }
            if (m_w != r_now) { l_w *= ex2_approx(m_w - r_now); m_w = r_now; }   // first use: l_w = 0, exp2(-inf) = 0
            // P = exp2(s * scale - R_i): one FFMA + one MUFU per element, packed bf16 pairs over S's own columns
            const uint64_t neg_m2 = pack2(-r_now, -r_now), scale2 = pack2(a.scale_log2, a.scale_log2);
            uint64_t part2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
            uint32_t pk[4][16];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    float x0, x1;
                    unpack2(fma2(pack2(s[c][2 * e], s[c][2 * e + 1]), scale2, neg_m2), x0, x1);
                    const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                    part2[e & 1] = add2(part2[e & 1], pack2(p0, p1));
                    pk[c][e] = pack_bf16(p0, p1);
                }
            }
            if (!p_free) {      // the one P buffer is free once P V of step i-1 (the other group's) has read it
                ok = mbar_wait_warp(bar_pvdone(wg ^ 1), uint32_t((i - 1) >> 1) & 1u, abortp, 0, limit);
                if (!ok) { if (lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 12, i, blockIdx.x); break; }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_st16(tP + c * 16, pk[c]);
            {
                float s0, s1, s2, s3;
                unpack2(part2[0], s0, s1); unpack2(part2[1], s2, s3);
                l_w += (s0 + s1) + (s2 + s3);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive_warp(bar_pfull(wg));
        }
        // combine the two groups' sums under the final reference (the later step holds the larger one)
        if (ok) {
            fin[wg][0][r_loc] = m_w;
            fin[wg][1][r_loc] = l_w;
            mbar_arrive_warp(bar_fin(quarter));
            ok = mbar_wait_warp(bar_fin(quarter), 0, abortp, 0, limit);
            if (!ok && lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 11, T, blockIdx.x);
        }
        if (ok) {
            ok = mbar_wait_warp(bar_o, 0, abortp, 20, limit);
            if (!ok && lane == 0) set_status(a.hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 8, T, blockIdx.x);
        }
        if (ok) {
            tc_fence_after();
            const float m0 = fin[0][0][r_loc], m1 = fin[1][0][r_loc];
            const float r_fin = fmaxf(m0, m1);
            const float l_tot = fin[0][1][r_loc] * ex2_approx(m0 - r_fin) + fin[1][1][r_loc] * ex2_approx(m1 - r_fin);
            const float inv = 1.f / l_tot;
            // each group writes half of the head dimension
            __nv_bfloat16* op = a.O + b * a.os[0] + h * a.os[1] + int64_t(row) * a.os[2] + wg * (D / 2);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                float o[32];
                tmem_ld32(tmem + lane_base + kColO + wg * (D / 2) + c * 32, o);      // warp-collective: every lane takes part
                tmem_wait_ld();
                if (row < a.N) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 u;
                        u.x = pack_bf16(o[8 * v + 0] * inv, o[8 * v + 1] * inv);
                        u.y = pack_bf16(o[8 * v + 2] * inv, o[8 * v + 3] * inv);
                        u.z = pack_bf16(o[8 * v + 4] * inv, o[8 * v + 5] * inv);
                        u.w = pack_bf16(o[8 * v + 6] * inv, o[8 * v + 7] * inv);
                        *reinterpret_cast<uint4*>(op + c * 32 + v * 8) = u;
                    }
                }
            }
            if (wg == 0 && row < a.N) a.LSE[bh * a.N + row] = (r_fin + log2f(l_tot)) * kLn2;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever arms, with the limit the caller gives,
// and must come back with CARNATOR_ERR_DEVICE_TIMEOUT in the header (same helpers as the kernels above).
__global__ void wait_timeout_selftest_kernel(WsHeader* hdr, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long bar_mem;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait_warp(bar, 0, &abort_flag, 50, limit_ns);
    if (!ok && threadIdx.x == 0) set_status(hdr, CARNATOR_ERR_DEVICE_TIMEOUT, 90, 0, 0);
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// 4-D map over a [B,H,N,D] bf16 tensor with arbitrary (16-byte multiple) strides: box = 64 x box_rows x 1 x 1,
// 128-byte swizzle, rows >= N read as zero.
inline bool make_map(CUtensorMap* map, const void* base, int B, int H, int N, int D, const int64_t st[3], int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {cuuint64_t(D), cuuint64_t(N), cuuint64_t(H), cuuint64_t(B)};
    // the stride of a size-1 axis is never used for addressing but must still be a valid value; a zero stride on a
    // longer axis cannot be expressed (callers check tma_strides_ok before they get here)
    const cuuint64_t row = cuuint64_t(st[2]) * 2;
    if ((H > 1 && st[1] <= 0) || (B > 1 && st[0] <= 0)) return false;
    const cuuint64_t s_h = st[1] > 0 ? cuuint64_t(st[1]) * 2 : row * N;
    const cuuint64_t s_b = st[0] > 0 ? cuuint64_t(st[0]) * 2 : s_h * H;
    cuuint64_t strides[3] = {row, s_h, s_b};
    cuuint32_t box[4] = {64, cuuint32_t(box_rows), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same tensor with the head dimension split into its 64-element halves as a dimension of its own, behind the
// tokens: one box = D/64 halves x box_rows tokens x 64 elements lands in shared memory as [half][token][64] (each
// half a 128-byte-swizzled slab), so one copy fetches what make_map's boxes fetch in D/64.
inline bool make_map_halves(CUtensorMap* map, const void* base, int B, int H, int N, int D, const int64_t st[3], int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {64, cuuint64_t(N), cuuint64_t(D / 64), cuuint64_t(H), cuuint64_t(B)};
    const cuuint64_t row = cuuint64_t(st[2]) * 2;
    if ((H > 1 && st[1] <= 0) || (B > 1 && st[0] <= 0)) return false;
    const cuuint64_t s_h = st[1] > 0 ? cuuint64_t(st[1]) * 2 : row * N;
    const cuuint64_t s_b = st[0] > 0 ? cuuint64_t(st[0]) * 2 : s_h * H;
    cuuint64_t strides[4] = {row, 128, s_h, s_b};
    cuuint32_t box[5] = {64, cuuint32_t(box_rows), cuuint32_t(D / 64), 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 2-D map over a row-major [rows, D] bf16 array: box = box_cols x box_rows (64 columns: 128-byte swizzle, 32 columns:
// 64-byte swizzle), rows past the end read as zero.
inline bool make_map_2d(CUtensorMap* map, const void* base, int64_t rows, int D, int box_rows, int box_cols = 64) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cuuint64_t(D), cuuint64_t(rows)};
    cuuint64_t strides[1] = {cuuint64_t(D) * 2};
    cuuint32_t box[2] = {cuuint32_t(box_cols), cuuint32_t(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace tc

// A tensor map cannot express a zero stride, so a tensor that is shared over heads or batch entries (stride 0 on an
// axis longer than 1) is not read through TMA: such shapes run on the portable kernel.
inline bool tma_strides_ok(const carnator_shape* s, const int64_t st[3]) {
    return (s->B == 1 || st[0] > 0) && (s->H == 1 || st[1] > 0);
}

inline bool tcgen05_supported(const carnator_shape* s) {
    return s->block_q == tc::kBlock && s->block_k == tc::kBlock && (s->D == 64 || s->D == 128) &&
           tma_strides_ok(s, s->k_stride) && tma_strides_ok(s, s->v_stride);
}

template <int D>
inline carnator_status launch_tc(const AttnArgs& a, const CUtensorMap& mk, const CUtensorMap& mv,
                                 cudaStream_t stream, char* err, size_t errlen) {
    using C = tc::Cfg<D>;
    auto kern = tc::attn_tcgen05_kernel<D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(C::kSmemBytes));
    if (e != cudaSuccess) { snprintf(err, errlen, "cudaFuncSetAttribute(tcgen05): %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    // The register hand-over inside the kernel only completes if the CTA owns enough registers: check what the
    // compiler allocated instead of finding out on the device.
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) { snprintf(err, errlen, "cudaFuncGetAttributes(tcgen05): %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    if (fa.numRegs * tc::kThreads < tc::kSoftmaxWarps * 32 * tc::kRegsSoftmax + 128 * tc::kRegsService) {
        snprintf(err, errlen, "attn_tcgen05_kernel was built with %d registers per thread: too few for its setmaxnreg split", fa.numRegs);
        return CARNATOR_ERR_UNSUPPORTED;
    }
    dim3 grid(a.nqb, a.H, a.B);
    kern<<<grid, tc::kThreads, C::kSmemBytes, stream>>>(mk, mv, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(err, errlen, "attn_tcgen05_kernel: %s", cudaGetErrorString(e)); return CARNATOR_ERR_CUDA; }
    return CARNATOR_OK;
}

inline carnator_status launch_tcgen05(const AttnArgs& a, const carnator_shape* s, cudaStream_t stream,
                                      char* err, size_t errlen, long long* launches) {
    CUtensorMap mk, mv;      // Q is read with plain loads (once per CTA, into tensor memory)
    if (!tc::make_map(&mk, a.K, a.B, a.H, a.N, s->D, a.ks, tc::kBlock) ||
        !tc::make_map(&mv, a.V, a.B, a.H, a.N, s->D, a.vs, tc::kBlock)) {
        snprintf(err, errlen, "cuTensorMapEncodeTiled failed or is unavailable");
        return CARNATOR_ERR_CUDA;
    }
    carnator_status st = (s->D == 128) ? launch_tc<128>(a, mk, mv, stream, err, errlen)
                                       : launch_tc<64>(a, mk, mv, stream, err, errlen);
    if (st == CARNATOR_OK) *launches = 1;
    return st;
}

}  // namespace carnator
