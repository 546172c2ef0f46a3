// Attention-JVP forward kernel for sm_100a (Algorithm 2: FlashAttention-2 forward with JVP).
//
// One CTA owns a 128-row query tile of one (batch, head) and streams the keys in
// tiles of 64 (128 in the forward-only mode); CTAs are persistent (one per SM) and walk the query tiles round-robin, so that the epilogue of
// one tile overlaps the loads and the first score MMAs of the next.  Roles (warp-specialised, 384 threads, laid
// out by warpgroup so that each can have its own register budget):
//   warp 0      MMA issuer: the whole warp runs the loop in lock step, one elected lane's tcgen05.mma take effect,
//               with accumulators in tensor memory.
//   warp 1      TMA producer: Q,tQ per query tile, K|tK and V|tV tiles into a shared-memory ring.  (Warps 2, 3 idle.)
//   warps 4-7   softmax: thread (w, lane) owns query row 32*(w%4) + lane (its tensor-memory lane) and
//               all columns of every score tile.  Reads S and tS from tensor memory, keeps m, l, r
//               (Algorithm 2 lines 10-12, 16) in registers, writes P~ and H~ = P~ . tS back to tensor
//               memory as bf16 MMA operands, and rescales the accumulators when the running max moves.
//   warps 8-11  a second softmax group on alternate key tiles, or (one group) the epilogue warps, which run
//               lines 19-23 for every finished query tile while the softmax warps are in the next one.
//
// Tensor-memory map (512 columns x 128 lanes, fp32):
//   [0, D)        O  accumulator (line 13)
//   [D, 2D)       T = A + B accumulator (lines 14 and 18 share one accumulator, since only
//                 A + B is ever used, line 22)
//   [c0+128b, +64)     S  of score buffer b; P~ (bf16) overwrites it
//   [c0+64+128b, +64)  tS of score buffer b; H~ (bf16) overwrites it
// Two score buffers from column c0 = 256 (tile g uses buffer g % 2), or, where the accumulators need no more than
// 128 columns (D = 64, and the forward-only mode), three from c0 = 128: the score MMAs then run three tiles
// ahead of the value MMAs, which takes the round trip tensor pipe -> softmax warps -> tensor pipe out of the
// tile period.
//
// Contractions per key tile (line 9 and lines 13, 14, 18):
//   [S | Q tK^T] = Q [K ; tK]^T      one MMA chain, N = 128 (K and tK tiles are stacked in smem)
//   tS          += tQ K^T            N = 64
//   [O | T]     += P~ [V | tV]       A operand from tensor memory, N = 2D
//   T           += H~ V              N = D
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace attn_jvp {

constexpr int kBlockM = 128;        // query rows per CTA (B_r)
constexpr int kBlockN = 64;         // keys per tile (B_c) ...
constexpr int kSoftmaxThreads = 128;   // four softmax warps per group: one thread per query row
constexpr int kMmaWarp = 0;            // the two single-thread roles come first (oldest warps of the CTA)
constexpr int kProducerWarp = 1;
// The roles are laid out by warpgroup, so that each can be given its own register budget (384 threads):
// warps 0..3 = MMA, producer and two idle warps; warps 4..7 = softmax group 0; warps 8..11 = softmax group 1 (two
// groups take alternate key tiles), or, with one softmax group, the epilogue warps: they run the epilogue of every
// work item (normalise, round, stage the output tiles), so that the softmax warps go straight on to the next item's
// first key tile.  With two groups the group that finishes an item runs its epilogue while the other is already in
// the next item.
__host__ __device__ constexpr int first_softmax_warp(int) { return 4; }
__host__ __device__ constexpr int num_threads(int) { return 3 * kSoftmaxThreads; }
constexpr int kRegsLightWarps = 104;    // registers per thread of warps 0..3 ...
constexpr int kRegsSoftmaxWarps = 200; // ... and of warps 4..11 (128 * 104 + 256 * 200 <= 384 * 168 = 64512)
constexpr int kTmemCols = 512;
constexpr int kScoreBufStride = 128; // tensor-memory columns of one score buffer {S 64, tS 64}
constexpr float kRescaleThreshold = 8.0f;   // log2 units: rescale only when the max grows by > 2^8
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // bound on every device-side wait
constexpr uint32_t kTryWaitHintNs = 20000u;   // a waiting thread may sleep this long per try (it is woken on completion)

enum Mode : int { kModeJvp = 0, kModeKvTangentFree = 1, kModeFwdOnly = 2 };

// Optional in-kernel timeline (compile with -DATTN_JVP_TRACE; never part of the shipped library):
// one CTA stamps clock64() at the hand-over points of its roles for the first kTraceSteps key tiles.
#ifdef ATTN_JVP_TRACE
constexpr int kTraceSteps = 96;
constexpr int kTraceEvents = 32;
__device__ long long g_trace[kTraceEvents][kTraceSteps];
#if ATTN_JVP_TRACE >= 2
#define TRACE(evt, idx) do { if (trace_on && (idx) < kTraceSteps) g_trace[evt][idx] = clock64(); } while (0)
#else
#define TRACE(evt, idx) do { } while (0)     // level 1: only the CTA's begin / end stamps
#endif
#else
#define TRACE(evt, idx) do { } while (0)
#endif
// Totals per role (both trace levels): cycles spent blocked, summed in a register and written once at the end.
#ifdef ATTN_JVP_TRACE
#define ACC_DECL(v) long long v = 0, v##_n = 0
#define ACC_BEGIN(v) const long long v##_t0 = clock64()
#define ACC_END(v) do { v += clock64() - v##_t0; ++v##_n; } while (0)
#define ACC_WRITE(slot, v) do { if (trace_on && lane == 0) { g_trace[kTraceEvents - 2][2 * (slot)] = v; g_trace[kTraceEvents - 2][2 * (slot) + 1] = v##_n; } } while (0)
#else
#define ACC_DECL(v) do { } while (0)
#define ACC_BEGIN(v) do { } while (0)
#define ACC_END(v) do { } while (0)
#define ACC_WRITE(slot, v) do { } while (0)
#endif

// Set by any kernel whose bounded wait expired; later CTAs see it and leave at once.
__device__ int g_abort_flag = 0;
// Which wait expired first (diagnostics): shared-memory address of the barrier, the parity waited for,
// threadIdx.x and blockIdx.x; [4] is nonzero once filled.  Debug builds (-DATTN_JVP_DEBUG) also record
// the addresses of the kernel's barriers in g_barrier_layout so that the first word can be given a name.
__device__ unsigned g_timeout_info[5] = {0, 0, 0, 0, 0};
#ifdef ATTN_JVP_DEBUG
__device__ unsigned g_barrier_layout[32];
#endif

struct KernelArgs {
    __nv_bfloat16* o;
    __nv_bfloat16* to;
    float* lse;
    int* host_status;   // mapped pinned host word, receives the timeout code
    int H, Lq, Lk;
    int n_kv_tiles;     // key tiles (of the kernel variant's size) in all of Lk
    float scale;        // s
    float scale_log2;   // s * log2(e)
    // optional side output: mu = rowsum(P . tS) = d(LSE) along the tangent, fp32 [B][H][Lq] (may be null)
    float* mu;
    // split-KV mode: the keys are cut into `splits` chunks of `tiles_per_split` tiles; a work item is then one
    // (query tile, head, batch, chunk);
    // chunk s writes normalised partial results (fp32) instead of the final outputs
    int splits;
    int tiles_per_split;
    float* part_o;      // [splits][B][Lq][H][D]
    float* part_to;     // [splits][B][Lq][H][D]
    float* part_lse;    // [splits][B][H][Lq]
    float* part_mu;     // [splits][B][H][Lq]
    int B;
    int n_q_tiles;      // 128-row query tiles per (batch, head)
    int n_items;        // work items = n_q_tiles * H * B * splits; the grid's CTAs share them round-robin
};

// Shared-memory plan of a kernel variant.
//   One Q/tQ buffer (full JVP at D = 128, and every CTA-pair variant): Q, tQ resident, ring slots of one primal +
//   one tangent tile (= one 128 x D bf16 output tile, which is what the ring's staging slots rely on).
//   Two Q/tQ buffers (the variants that leave room: no K/V tangents, or D = 64): the next item's Q, tQ are loaded
//   while the current item runs, ring slots hold exactly what the mode loads, and an item's output tiles are staged
//   in its own Q/tQ buffer (dead once its last value MMAs are complete) instead of in ring slots.
// ... except in the forward-only mode (one CTA per query tile, no key chunks), which takes 128 keys per
// tile: there is no tS, so a score buffer of 128 tensor-memory columns holds S of 128 keys, the N = 128 score MMAs
// run at the pipe's full rate (64 cycles for twice the work of an N = 64 one at 54), and the per-tile costs of
// the issuing and softmax warps (barriers, tensor-memory round trips, bookkeeping) are paid half as often.
__host__ __device__ constexpr int key_tile(int D, int mode, bool split, bool pair) {
    return (mode == kModeFwdOnly && !split && !pair) ? 2 * kBlockN : kBlockN;
}

template <int D, int MODE, int kGroups, bool kPair, bool kSplit = false>
struct SmemPlan {
    static constexpr int kBN = key_tile(D, MODE, kSplit, kPair);   // keys per tile
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzle atoms per row
    static constexpr int kQHalfBytes = kBlockM * 128;      // 16 KB: 128 rows x 128 B
    static constexpr int kQBytes = kHalves * kQHalfBytes;
    static constexpr int kKvHalfBytes = kBN * 128;         // 8 KB: 64 rows x 128 B (16 KB with 128-key tiles)
    static constexpr bool kDoubleQ = kPair ? (MODE == kModeKvTangentFree) : (MODE != kModeJvp || D == 64);
    static constexpr int kQSets = kDoubleQ ? 2 : 1;
    static constexpr int kQSetBytes = (kDoubleQ && MODE == kModeFwdOnly) ? kQBytes : 2 * kQBytes;   // Q (+ tQ)
    static constexpr int kTilesPerSlot = (!kDoubleQ || MODE == kModeJvp) ? 2 : 1;                   // primal (+ tangent)
    static constexpr int kSlotBytes = kTilesPerSlot * kHalves * kKvHalfBytes;
    static constexpr int kRoom = 224 * 1024 - kQSets * kQSetBytes;
    static constexpr int kSlots = kDoubleQ ? (kRoom / kSlotBytes < 8 ? kRoom / kSlotBytes : 8) : ((D == 128) ? 5 : 8);
    static constexpr int kRingOffset = kQSets * kQSetBytes;
    static constexpr int kOperandBytes = kRingOffset + kSlots * kSlotBytes;
    // Four per-row fp32 values go through shared memory, placed after the operand tiles: two softmax groups exchange
    // the reference max, the centring constant of tS and their partial l and r; with one group the softmax warps
    // hand m, the centring constant, l and r of a finished item to the epilogue warps there.
    static constexpr int kExchangeBytes = 4 * kBlockM * 4;
    // The dynamic allocation is declared 1024-byte aligned (the operand tiles need that for the 128-byte
    // swizzle); static shared memory (barriers, a few words) stays below 1 KB, so that at D = 128 operands
    // (224 KB), exchange area (2 KB) and static part fill the 227 KB a CTA can have exactly.
    static constexpr int kDynBytes = kOperandBytes + kExchangeBytes;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kTryWaitHintNs) : "memory");
    return ok != 0;
}
// Non-blocking test of a phase (never suspends the thread).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Shared by all roles of a CTA: set once a wait gave up, so that the others stop waiting too.
struct AbortState {
    volatile int* cta_flag;   // shared memory
    int* host_status;
};

__device__ __noinline__ void report_device_error(const AbortState& st, int code) {
    *st.cta_flag = 1;
    atomicExch(&g_abort_flag, 1);
    if (st.host_status) {
        *reinterpret_cast<volatile int*>(st.host_status) = code;   // ATTN_JVP_ERR_DEVICE_*
        __threadfence_system();
    }
}

// Bounded wait: true when the phase completed, false when the CTA must abandon its tile.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const AbortState& st) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (*st.cta_flag) return false;
            if (globaltimer_ns() - t0 > kWaitLimitNs) {
                if (atomicCAS(&g_timeout_info[4], 0u, 1u) == 0u) {
                    g_timeout_info[0] = bar;
                    g_timeout_info[1] = parity;
                    g_timeout_info[2] = threadIdx.x;
                    g_timeout_info[3] = blockIdx.x;
                }
                report_device_error(st, 10);   // ATTN_JVP_ERR_DEVICE_TIMEOUT
                return false;
            }
        }
    }
}

// The same for a whole warp whose lanes go on to warp-collective (.sync.aligned) instructions:
// every lane takes the same decision.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const AbortState& st) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, st));
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// Tile store shared -> global through a tensor map (rows beyond the tensor's extent are clipped).
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// The stores committed so far have read their shared-memory source (it may be overwritten).
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// The stores committed so far are complete.
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders this thread's shared-memory writes before later reads by the asynchronous proxy (TMA).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Brings a tile into L2 only.
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// True in exactly one lane of a fully active warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t is_leader;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(is_leader));
    return is_leader != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- CTA pair (cluster of two CTAs on the two SMs of a TPC, one tcgen05.mma feeding both) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrival on a barrier of another CTA of the cluster.  What is handed over with it lives in tensor memory and is
// ordered by the tcgen05 fences on both sides; a cluster-scope release on the arrival itself was measured to cost
// about a thousand cycles per arrival and is not needed for that.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_shared_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// Barrier over all threads of the cluster.  Every thread of both CTAs reaches each of its uses on every path
// (all other waits in the kernel are bounded), so it cannot be left waiting.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA tile load of a CTA pair: the data lands in this CTA's shared memory, the bytes are counted on a barrier that
// may live in the pair's other CTA (`bar` is a shared::cluster address).  No multicast: each CTA fetches its own.
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// completion of all earlier MMAs of this thread, signalled on the barrier at this address in BOTH CTAs of the pair
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}
template <bool kAccumulate>
__device__ __forceinline__ void mma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    if (kAccumulate) {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, 1, 1;\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
    }
}
__device__ __forceinline__ void mma_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// The same instructions guarded by a per-lane predicate: the issuing warp stays converged (every lane executes the
// instruction stream, the elected lane alone issues), which keeps its loop out of divergent-branch handling.
template <bool kAccumulate, bool kPairMma>
__device__ __forceinline__ void mma_ss_if(uint32_t pred, uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    if (kPairMma) {
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %4, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "@q tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(pred), "r"(kAccumulate ? 1u : 0u) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %4, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(pred), "r"(kAccumulate ? 1u : 0u) : "memory");
    }
}
template <bool kPairMma>
__device__ __forceinline__ void mma_ts_if(uint32_t pred, uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    if (kPairMma) {
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %5, 0;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "@q tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(pred) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %5, 0;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(pred) : "memory");
    }
}
template <bool kPairMma>
__device__ __forceinline__ void tc_commit_if(uint32_t pred, uint32_t bar) {
    if (kPairMma) {
        asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t"
                     "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
                     ::"r"(bar), "h"(static_cast<uint16_t>(3)), "r"(pred) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
                     "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                     ::"r"(bar), "r"(pred) : "memory");
    }
}

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major, int m = kBlockM) {
    return (1u << 4)                       // accumulator format: fp32
         | (1u << 7)                       // A format: bf16
         | (1u << 10)                      // B format: bf16
         | (0u << 15)                      // A: K-major
         | ((b_mn_major ? 1u : 0u) << 16)  // B: K-major or MN-major
         | (static_cast<uint32_t>(n >> 3) << 17)
         | (static_cast<uint32_t>(m >> 4) << 24);
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (rows x 64 bf16 per swizzle atom): lbo unused.
//   MN-major operand (64 contiguous bf16 along N per atom): lbo = bytes between N atoms.
// The high word is a constant; the low word holds (address >> 4) and (lbo >> 4) << 16, so moving
// along an operand is one 32-bit add of (byte offset >> 4) -- the issuing thread does nothing else
// per instruction.
constexpr uint32_t kDescHi = (1024u >> 4)      // stride between 8-row groups
                           | (1u << 14)        // descriptor version for sm_100
                           | (2u << 29);       // SWIZZLE_128B
__device__ __forceinline__ uint32_t make_desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}

// Full 64-bit descriptor from its low word.
__device__ __forceinline__ uint64_t make_desc(uint32_t lo) {
    uint64_t d;
    asm volatile("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(kDescHi));
    return d;
}
// D[tmem] (+)= A[smem] * B[smem]; the accumulate flag is a compile-time choice so that nothing but the
// MMA itself has to be issued per instruction.
template <bool kAccumulate>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    if (kAccumulate) {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
    } else {
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, 1, 1;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
    }
}
// D[tmem] (+)= A[tmem] * B[smem]; runtime accumulate flag (the first value MMA of a query tile overwrites)
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 lanes x 32 columns: thread t of the warp receives columns [addr.col, +32) of lane (warp%4)*32 + t
// into v[o .. o+31].
#define TMEM_LD32(addr, v, o)                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                  \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                  \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];" \
                 : "=r"(v[(o) + 0]), "=r"(v[(o) + 1]), "=r"(v[(o) + 2]), "=r"(v[(o) + 3]), "=r"(v[(o) + 4]), "=r"(v[(o) + 5]), "=r"(v[(o) + 6]), "=r"(v[(o) + 7]), "=r"(v[(o) + 8]), "=r"(v[(o) + 9]), "=r"(v[(o) + 10]), "=r"(v[(o) + 11]), "=r"(v[(o) + 12]), "=r"(v[(o) + 13]), "=r"(v[(o) + 14]), "=r"(v[(o) + 15]), "=r"(v[(o) + 16]), "=r"(v[(o) + 17]), "=r"(v[(o) + 18]), "=r"(v[(o) + 19]), "=r"(v[(o) + 20]), "=r"(v[(o) + 21]), "=r"(v[(o) + 22]), "=r"(v[(o) + 23]), "=r"(v[(o) + 24]), "=r"(v[(o) + 25]), "=r"(v[(o) + 26]), "=r"(v[(o) + 27]), "=r"(v[(o) + 28]), "=r"(v[(o) + 29]), "=r"(v[(o) + 30]), "=r"(v[(o) + 31])          \
                 : "r"(addr) : "memory")

#define TMEM_ST32(addr, v, o)                                                              \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                            \
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"                 \
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"        \
                 ::"r"(addr), "r"(v[(o) + 0]), "r"(v[(o) + 1]), "r"(v[(o) + 2]), "r"(v[(o) + 3]), "r"(v[(o) + 4]), "r"(v[(o) + 5]), "r"(v[(o) + 6]), "r"(v[(o) + 7]), "r"(v[(o) + 8]), "r"(v[(o) + 9]), "r"(v[(o) + 10]), "r"(v[(o) + 11]), "r"(v[(o) + 12]), "r"(v[(o) + 13]), "r"(v[(o) + 14]), "r"(v[(o) + 15]), "r"(v[(o) + 16]), "r"(v[(o) + 17]), "r"(v[(o) + 18]), "r"(v[(o) + 19]), "r"(v[(o) + 20]), "r"(v[(o) + 21]), "r"(v[(o) + 22]), "r"(v[(o) + 23]), "r"(v[(o) + 24]), "r"(v[(o) + 25]), "r"(v[(o) + 26]), "r"(v[(o) + 27]), "r"(v[(o) + 28]), "r"(v[(o) + 29]), "r"(v[(o) + 30]), "r"(v[(o) + 31])      \
                 : "memory")

#define TMEM_ST16(addr, v, o)                                                              \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "                            \
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"                \
                 ::"r"(addr), "r"(v[(o) + 0]), "r"(v[(o) + 1]), "r"(v[(o) + 2]), "r"(v[(o) + 3]), "r"(v[(o) + 4]), "r"(v[(o) + 5]), "r"(v[(o) + 6]), "r"(v[(o) + 7]), "r"(v[(o) + 8]), "r"(v[(o) + 9]), "r"(v[(o) + 10]), "r"(v[(o) + 11]), "r"(v[(o) + 12]), "r"(v[(o) + 13]), "r"(v[(o) + 14]), "r"(v[(o) + 15])      \
                 : "memory")

__device__ __forceinline__ void tmem_st2(uint32_t addr, float a, float b) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};"
                 ::"r"(addr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)) : "memory");
}
__device__ __forceinline__ void tmem_ld2(uint32_t addr, float& a, float& b) {
    uint32_t x, y;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(addr) : "memory");
    a = __uint_as_float(x);
    b = __uint_as_float(y);
}

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Two fp32 lanes per instruction (sm_100 packed fp32 arithmetic): halves the FMA-pipe instruction count
// of the softmax inner loops.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
// Score buffers a kernel variant can have (see the tensor-memory map above).
__host__ __device__ constexpr int score_buffers(int D, int mode) {
    return ((mode == kModeFwdOnly ? D : 2 * D) <= 128) ? 3 : 2;
}

// kPair: the kernel is launched in clusters of two CTAs that share every work item -- a 256-row query block of
// which each CTA owns 128 rows (its own Q, tQ, softmax warps, accumulators and outputs).  The MMA warp of the
// cluster's first CTA issues every tcgen05.mma for both (cta_group::2, M = 256): the B operands (K, tK, V, tV
// tiles) are split between the two CTAs' shared memories, each CTA loading its part through its own TMA
// requests (no multicast), and one instruction stream feeds two tensor pipes.  tm_k32 (32-row boxes of K) is
// only used by that variant.
template <int D, int MODE, bool kSplit, int kGroups, bool kPair>
__global__ void __launch_bounds__(num_threads(kGroups), 1)
attn_jvp_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_tq,
                    const __grid_constant__ CUtensorMap tm_tk, const __grid_constant__ CUtensorMap tm_tv,
                    const __grid_constant__ CUtensorMap tm_o, const __grid_constant__ CUtensorMap tm_to,
                    const __grid_constant__ CUtensorMap tm_k32, const KernelArgs args) {
    static_assert(!kPair || (D == 128 && !kSplit), "the CTA-pair variant exists at D = 128, without key chunks");
    using Plan = SmemPlan<D, MODE, kGroups, kPair, kSplit>;
    constexpr int kBN = Plan::kBN;                           // keys per tile
    constexpr bool kDoubleQ = Plan::kDoubleQ;
    constexpr int kFirstSoftmaxWarp = first_softmax_warp(kGroups);
    constexpr int kHalves = Plan::kHalves;
    constexpr int kSlots = Plan::kSlots;
    constexpr bool kHasTQ = (MODE != kModeFwdOnly);          // tS and T exist
    constexpr bool kHasTKV = (MODE == kModeJvp);             // tK, tV are read
    // The bf16 output tiles leave through shared memory and TMA stores: at the end of every item the ring gives
    // up one slot per output tensor (a slot is exactly one 128 x D bf16 tile).  The split-KV kernel writes its
    // fp32 partial results straight from registers and stages nothing.
    constexpr int kStageSlots = kSplit ? 0 : (kHasTQ ? 2 : 1);       // output tiles staged per item ...
    constexpr int kRingStage = kDoubleQ ? 0 : kStageSlots;           // ... of which in ring slots (else in the item's Q/tQ buffer)
    // P~ and H~ of a tile are handed to the MMA warp together (one barrier): the softmax warps form both in one
    // pass over the columns, so an earlier hand-over of P~ alone would gain nothing.
    constexpr int kBufs = score_buffers(D, MODE);            // score buffers = how many tiles the score MMAs run ahead
    constexpr int kScoreCol0 = (kBufs == 3) ? 128 : 256;     // first column of score buffer 0
    static_assert(kScoreCol0 + kBufs * kScoreBufStride <= kTmemCols, "score buffers must fit into tensor memory");
    static_assert((kHasTQ ? 2 * D : D) <= kScoreCol0, "accumulators and score buffers overlap");
    static_assert(kDoubleQ || Plan::kSlotBytes == Plan::kQBytes, "an output tile must fill one ring slot");

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q_full[2];  // Q, tQ of a work item are in shared memory (one barrier per Q/tQ buffer)
    __shared__ __align__(8) uint64_t bar_q_free;     // every score MMA of the item has completed: Q, tQ may be replaced
    __shared__ __align__(8) uint64_t bar_slot_full[kSlots];
    __shared__ __align__(8) uint64_t bar_slot_empty[kSlots];
    __shared__ __align__(8) uint64_t bar_s_full[kBufs];
    __shared__ __align__(8) uint64_t bar_p_full[kBufs];     // P~ and H~ of the tile are in tensor memory
    __shared__ __align__(8) uint64_t bar_pv_done[2];        // the value MMAs of tile g (and all before) are complete: [g & 1]
    __shared__ __align__(8) uint64_t bar_acc_free;   // the epilogue has read O and T: the next item may overwrite them
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ __align__(8) uint64_t bar_stage_ready;   // the item's staging slots are free of operand reads
    __shared__ __align__(8) uint64_t bar_stage_full;    // the softmax warps have written the item's output tiles
    // one barrier per quarter of the rows (a pair of warps: one of each softmax group, or softmax and epilogue warp):
    __shared__ __align__(8) uint64_t bar_m[4];          // two groups: the reference max after tile g is published (phase g & 1)
    __shared__ __align__(8) uint64_t bar_fin[4];        // l, r (one group: also m, centring constant) of the item are published
    __shared__ __align__(8) uint64_t bar_fin_read[4];   // ... and have been read by the warp that finishes the item
    __shared__ uint32_t tmem_base_smem;
    __shared__ int cta_abort;

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);   // warp-uniform by construction
    const int lane = threadIdx.x & 31;
#ifdef ATTN_JVP_TRACE
    const bool trace_on = blockIdx.x == (kPair ? (gridDim.x / 4) * 2 : gridDim.x / 2);
#endif

    // A CTA is persistent: it walks the work items blockIdx.x, blockIdx.x + gridDim.x, ... in the same order in
    // every role.  An item is one 128-row query tile of one (batch, head[, key chunk]); query tiles vary fastest
    // so that the CTAs running at one time share one head's K/V in L2.
    // CTA pair: both CTAs walk the same items (one item = two query tiles); this CTA's rank picks its rows.
    const uint32_t cta_rank = kPair ? cluster_ctarank() : 0u;
    const bool lead_cta = cta_rank == 0u;
    const int first_item = kPair ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int item_stride = kPair ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    struct Item { int q0, h, b, split, tile0, n_kv; };
    // Work item number -> (query tile, head, batch [, chunk]).  The roles walk their items with a fixed stride, so
    // after the first item the three indices are advanced by the stride's own decomposition (carry by compare and
    // subtract) instead of being divided out again: the divisions would sit on the critical path of every item
    // hand-over, once per role.
    struct Walk { int qt, h, z; };
    auto walk_init = [&](int item) -> Walk {
        Walk k;
        k.qt = item % args.n_q_tiles;
        const int rest = item / args.n_q_tiles;
        k.h = rest % args.H;
        k.z = rest / args.H;
        return k;
    };
    const Walk walk_stride = walk_init(item_stride);
    auto walk_step = [&](Walk& k) {
        k.qt += walk_stride.qt;
        if (k.qt >= args.n_q_tiles) { k.qt -= args.n_q_tiles; ++k.h; }
        k.h += walk_stride.h;
        if (k.h >= args.H) { k.h -= args.H; ++k.z; }
        k.z += walk_stride.z;
    };
    auto item_of = [&](const Walk& k) -> Item {
        Item w;
        w.q0 = k.qt * (kPair ? 2 * kBlockM : kBlockM) + static_cast<int>(cta_rank) * kBlockM;
        w.h = k.h;
        w.b = kSplit ? k.z / args.splits : k.z;
        w.split = kSplit ? k.z % args.splits : 0;
        w.tile0 = kSplit ? w.split * args.tiles_per_split : 0;       // first key tile of this item
        w.n_kv = kSplit ? min(args.tiles_per_split, args.n_kv_tiles - w.tile0) : args.n_kv_tiles;
        return w;
    };
    const int n_items = args.n_items;
    // Two Q/tQ buffers, no key chunks (every item then has the same number of key tiles): the key tiles of all of a
    // CTA's items form one stream.  The score MMAs of an item's leading tiles are issued in the last bursts of the
    // item before (its Q, tQ are resident by then), and the ring carries their K tiles in that order, so that an
    // item boundary costs the MMA warp and the producer nothing.
    const bool stream_items = kDoubleQ && !kSplit && args.n_kv_tiles >= kBufs;
    // Score buffer and barrier phase of a key tile, g % kBufs and (g / kBufs) & 1, carried along tile by tile (a
    // division by three per use would sit on the MMA warp's critical chain of dependent instructions).
    struct BufPos { int buf; uint32_t phase; };
    auto next_buf = [](BufPos& p) { if (++p.buf == kBufs) { p.buf = 0; p.phase ^= 1u; } };

    // An earlier CTA of this (or a previous) launch gave up: do not start.  One thread reads
    // the flag so that the whole CTA takes the same decision.
    // (A CTA pair takes this decision together, after its barriers are set up: see below.)
    if (!kPair) {
        if (threadIdx.x == 0) cta_abort = *reinterpret_cast<volatile int*>(&g_abort_flag);
        __syncthreads();
        if (cta_abort != 0) return;
    }

#ifdef ATTN_JVP_TRACE
    if (trace_on && threadIdx.x == 0) g_trace[kTraceEvents - 1][0] = clock64();      // CTA begins
#endif
    const uint32_t smem_base = smem_u32(smem_raw);
    // Q/tQ buffer of item number `it`, its `full` barrier and that barrier's phase
    auto q_addr = [&](int it) -> uint32_t { return smem_base + (kDoubleQ ? (it & 1) * Plan::kQSetBytes : 0); };
    auto tq_addr = [&](int it) -> uint32_t { return q_addr(it) + Plan::kQBytes; };
    auto q_full_bar = [&](int it) -> uint32_t { return smem_u32(&bar_q_full[kDoubleQ ? (it & 1) : 0]); };
    auto q_full_phase = [](int it) -> uint32_t { return static_cast<uint32_t>(kDoubleQ ? (it >> 1) : it) & 1u; };
    const uint32_t smem_ring = smem_base + Plan::kRingOffset;

    AbortState abort_state{&cta_abort, args.host_status};

    // The operand tiles need 1024-byte alignment (the dynamic allocation is declared that way) and the host
    // must have asked for the whole layout: this check keeps a mismatch from becoming a wrong or out-of-bounds
    // access.
    {
        uint32_t dyn_size;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_size));
        if ((smem_base & 1023u) != 0u || static_cast<uint32_t>(Plan::kDynBytes) > dyn_size) {
            if (threadIdx.x == 0) report_device_error(abort_state, 11);   // ATTN_JVP_ERR_DEVICE_LAYOUT
            return;
        }
    }

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar_q_full[0]), 1);
        mbar_init(smem_u32(&bar_q_full[1]), 1);
        mbar_init(smem_u32(&bar_q_free), 1);
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(smem_u32(&bar_slot_full[i]), 1);
            mbar_init(smem_u32(&bar_slot_empty[i]), 1);
        }
        for (int i = 0; i < kBufs; ++i) {
            mbar_init(smem_u32(&bar_s_full[i]), 1);
            // one arrival per softmax warp of the tile's group (CTA pair: of both CTAs, on the first CTA's barrier)
            mbar_init(smem_u32(&bar_p_full[i]), (kPair ? 2 : 1) * kSoftmaxThreads / 32);
        }
        mbar_init(smem_u32(&bar_pv_done[0]), 1);
        mbar_init(smem_u32(&bar_pv_done[1]), 1);
        mbar_init(smem_u32(&bar_acc_free), (kPair ? 2 : 1) * kSoftmaxThreads / 32);
        mbar_init(smem_u32(&bar_drain), 1);
        mbar_init(smem_u32(&bar_stage_ready), 1);
        mbar_init(smem_u32(&bar_stage_full), kSoftmaxThreads / 32);
        for (int i = 0; i < 4; ++i) {
            mbar_init(smem_u32(&bar_m[i]), 1);
            mbar_init(smem_u32(&bar_fin[i]), 1);
            mbar_init(smem_u32(&bar_fin_read[i]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
#ifdef ATTN_JVP_DEBUG
        if (blockIdx.x == 0) {
            const void* named[] = {&bar_q_full[0], &bar_q_free, &bar_slot_full[0], &bar_slot_empty[0], &bar_s_full[0],
                                   &bar_p_full[0], &bar_p_full[0], &bar_pv_done[0], &bar_acc_free, &bar_drain,
                                   &bar_stage_ready, &bar_stage_full, &bar_m[0], &bar_fin[0]};
            for (int i = 0; i < 14; ++i) g_barrier_layout[i] = smem_u32(named[i]);
        }
#endif
    }
    if (kPair) {
        // The pair decides together whether to run at all (an earlier CTA gave up): the first CTA reads the flag
        // and writes it into both CTAs; the cluster barrier also makes both CTAs' barriers visible to each other
        // before anything arrives on them from the other side.
        if (threadIdx.x == 0 && lead_cta) {
            const int flag = *reinterpret_cast<volatile int*>(&g_abort_flag);
            cta_abort = flag;
            st_shared_cluster_u32(map_to_cta(smem_u32(&cta_abort), 1u), static_cast<uint32_t>(flag));
        }
        cluster_sync_all();
        if (*reinterpret_cast<volatile int*>(&cta_abort) != 0) return;
    }
    if (warp == kMmaWarp) {
        // (pair: the same warp of both CTAs allocates, each in its own SM's tensor memory; both get column 0)
        if (kPair) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&tmem_base_smem)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&tmem_base_smem)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    if (warp == kProducerWarp && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        if (kHasTQ) prefetch_tensormap(&tm_tq);
        if (kHasTKV) { prefetch_tensormap(&tm_tk); prefetch_tensormap(&tm_tv); }
        if (kStageSlots > 0) prefetch_tensormap(&tm_o);
        if (kStageSlots > 1) prefetch_tensormap(&tm_to);
        if (kPair) prefetch_tensormap(&tm_k32);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_base_smem);
    const uint32_t tmem_o = tmem;
    const uint32_t tmem_t = tmem + D;

    // Phases.  Key tiles are numbered g = 0, 1, 2, ... over ALL items of this CTA; tile g uses score buffer
    // g % kBufs, phase (g / kBufs) & 1 of bar_s_full / bar_p_full, and phase (g >> 1) & 1 of
    // bar_pv_done[g & 1] (two barriers, so that a wait for tile g - 1 cannot be mistaken for one two tiles on).  Item number `it` (0, 1, ...)
    // uses phase it & 1 of bar_q_full / bar_q_free / bar_acc_free / bar_stage_ready / bar_stage_full.  The
    // shared-memory ring runs on without a break; per item it hands out 2 n slots to K/V tiles and then
    // kStageSlots slots to the output tiles.

    // The warps of the first warpgroup need few registers (two of them are idle), the softmax warps hold a whole
    // row of scores and tangent scores each; the budgets are moved accordingly.
    // (The forward-only softmax with 64-key tiles needs fewer registers than the 168 every thread of a 384-thread CTA
    // starts with; with 128-key tiles a thread holds 128 scores.)
    constexpr bool kMoveRegs = kHasTQ || kBN > kBlockN;
    if (warp < kFirstSoftmaxWarp) {
    if (kMoveRegs) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLightWarps));
    if (warp == kProducerWarp) {
        // =====================================================================================
        // TMA producer.  Per item: Q, tQ (once the previous item's score MMAs are done), then the ring in
        // consumption order K0, K1, V0, K2, V1, ..., K(n-1), V(n-2), V(n-1) (two score buffers; with three the
        // K tiles run one more ahead: K0, K1, K2, V0, K3, V1, ...).
        // =====================================================================================
        if (lane == 0) {
            constexpr uint32_t kQTx = (kHasTQ ? 2u : 1u) * Plan::kQBytes;
            constexpr uint32_t kKTx = (kHasTKV ? 2u : 1u) * kHalves * Plan::kKvHalfBytes;
            constexpr uint32_t kVTx = kKTx;
            // CTA pair: the `full` barriers that count, the MMA-issuing warp's, are the first CTA's; both CTAs' loads
            // report their bytes there and the first CTA's producer announces the bytes of both.
            // bytes between the 64-column halves of a K slot: the tangent tile's half sits between them unless the
            // slot holds the primal tile alone (two Q/tQ buffers, no K/V tangents)
            constexpr uint32_t kKHalfStride = Plan::kTilesPerSlot * Plan::kKvHalfBytes;
            // pair: offset of the second operand region of a ring slot (the halves of K / V that the N = 64 and
            // N = 128 MMAs take from each CTA at a common offset)
            constexpr uint32_t kPairRegionB = kHalves * Plan::kKvHalfBytes;   // 16 KB at D = 128
            static_assert(!kPair || kPairRegionB == 16384, "pair layout is laid out for D = 128");
            // ring position: slot, the parity of the slot's `full` phase that this lap completes, and whether the
            // ring has been round once (before that the slots are empty without anybody saying so)
            int r_slot = 0;
            uint32_t r_parity = 0;
            bool r_lapped = false;
            bool ok = true;
            Item w{};
            // waits until the slot at the ring position is empty, hands it out and moves on
            auto acquire = [&](int& slot, uint32_t& slot_addr, uint32_t& bar) -> bool {
                slot = r_slot;
                if (r_lapped) {
                    if (!mbar_wait(smem_u32(&bar_slot_empty[slot]), r_parity ^ 1u, abort_state)) return false;
                }
                slot_addr = smem_ring + slot * Plan::kSlotBytes;
                bar = kPair ? map_to_cta(smem_u32(&bar_slot_full[slot]), 0u) : smem_u32(&bar_slot_full[slot]);
                TRACE(0, slot);       // producer: slot acquired, loads issued next
                if (++r_slot == kSlots) { r_slot = 0; r_parity ^= 1u; r_lapped = true; }
                return true;
            };
            auto load_k = [&](int j) -> bool {
                int slot;
                uint32_t dst, bar;
                if (!acquire(slot, dst, bar)) return false;
                if (kPair) {
                    // With K/V tangents the stacked operand [K ; tK] is split by tensor: this CTA holds K (first CTA)
                    // or tK (second) as [half 0 (8 KB)][half 1 (8 KB)], and the N = 64 operand of tQ K^T is split by
                    // rows: K rows 32 r .. 32 r + 31 as [half 0 (4 KB)][half 1 (4 KB)] in the slot's second region.
                    // Without them every score MMA has N = 64 and takes that row split alone, from the slot's start.
                    constexpr uint32_t kTxPerCta = (kHasTKV ? 2 * Plan::kKvHalfBytes : 0) + Plan::kKvHalfBytes;
                    constexpr uint32_t kRows32Off = kHasTKV ? kPairRegionB : 0;
                    if (lead_cta) mbar_arrive_expect_tx(smem_u32(&bar_slot_full[slot]), 2 * kTxPerCta);
                    const int row0 = (w.tile0 + j) * kBN;
#pragma unroll
                    for (int hf = 0; hf < kHalves; ++hf) {
                        if (kHasTKV)
                            tma_load_4d_pair(dst + hf * Plan::kKvHalfBytes, lead_cta ? &tm_k : &tm_tk, bar, hf * 64, w.h, row0, w.b);
                        tma_load_4d_pair(dst + kRows32Off + hf * (Plan::kKvHalfBytes / 2), &tm_k32, bar, hf * 64, w.h,
                                         row0 + 32 * static_cast<int>(cta_rank), w.b);
                    }
                    return true;
                }
                mbar_arrive_expect_tx(bar, kKTx);
                // per 64-column half: [K_half (8 KB)][tK_half (8 KB)] so that [K ; tK] is one N = 128 operand
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_4d(dst + hf * kKHalfStride, &tm_k, bar, hf * 64, w.h, (w.tile0 + j) * kBN, w.b);
                    if (kHasTKV)
                        tma_load_4d(dst + hf * kKHalfStride + Plan::kKvHalfBytes, &tm_tk, bar, hf * 64, w.h, (w.tile0 + j) * kBN, w.b);
                }
                return true;
            };
            auto load_v = [&](int j) -> bool {
                int slot;
                uint32_t dst, bar;
                if (!acquire(slot, dst, bar)) return false;
                if (kPair) {
                    // With K/V tangents [V | tV] is split by tensor: this CTA holds V (first CTA) or tV (second) as two
                    // 64-wide N atoms, and the N = 128 operand of H~ V is split by columns: V atom r in the slot's
                    // second region.  Without them every value MMA has N = 128 and takes that column split alone.
                    constexpr uint32_t kTxPerCta = (kHasTKV ? 2 * Plan::kKvHalfBytes : 0) + Plan::kKvHalfBytes;
                    constexpr uint32_t kAtomOff = kHasTKV ? kPairRegionB : 0;
                    if (lead_cta) mbar_arrive_expect_tx(smem_u32(&bar_slot_full[slot]), 2 * kTxPerCta);
                    const int row0 = (w.tile0 + j) * kBN;
                    if (kHasTKV) {
#pragma unroll
                        for (int hf = 0; hf < kHalves; ++hf)
                            tma_load_4d_pair(dst + hf * Plan::kKvHalfBytes, lead_cta ? &tm_v : &tm_tv, bar, hf * 64, w.h, row0, w.b);
                    }
                    tma_load_4d_pair(dst + kAtomOff, &tm_v, bar, 64 * static_cast<int>(cta_rank), w.h, row0, w.b);
                    return true;
                }
                mbar_arrive_expect_tx(bar, kVTx);
                // [V_half0][V_half1][tV_half0][tV_half1]: consecutive 64-wide N atoms of [V | tV]
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_4d(dst + hf * Plan::kKvHalfBytes, &tm_v, bar, hf * 64, w.h, (w.tile0 + j) * kBN, w.b);
                    if (kHasTKV)
                        tma_load_4d(dst + (kHalves + hf) * Plan::kKvHalfBytes, &tm_tv, bar, hf * 64, w.h, (w.tile0 + j) * kBN, w.b);
                }
                return true;
            };
            // Output tiles of the item before: staged by the softmax warps in `stage_slot[]`, stored from here.
            bool stage_pending = false;
            int stage_slot[2] = {0, 0};
            int stage_it = 0;
            Item stage_w{};
            // In two steps where the staging buffers are the item's Q/tQ buffers: the stores are issued as soon as the
            // staged tiles are seen complete (`only_if_ready`: without waiting for them), and what needs their
            // shared-memory reads to be over -- the load of the next item's Q, tQ into that buffer -- comes a tile
            // later, so that this thread keeps the ring filled meanwhile instead of sitting in the wait.
            bool stores_in_flight = false;
            auto store_staged_finish = [&]() {
                tma_store_wait_read();
                TRACE(18, stage_it);  // producer: staging buffers read
                stores_in_flight = false;
            };
            auto store_staged = [&](bool only_if_ready = false, bool finish = true) -> bool {
                if (only_if_ready) {
                    if (!mbar_test_wait(smem_u32(&bar_stage_full), stage_it & 1)) return true;
                } else if (!mbar_wait(smem_u32(&bar_stage_full), stage_it & 1, abort_state)) {
                    return false;
                }
                TRACE(17, stage_it);  // producer: staged tiles complete, stores issued next
                // staged in two ring slots, or (two Q/tQ buffers) in the item's own Q and tQ buffer
                const uint32_t src_o = kDoubleQ ? q_addr(stage_it) : smem_ring + stage_slot[0] * Plan::kSlotBytes;
                const uint32_t src_t = kDoubleQ ? tq_addr(stage_it) : smem_ring + stage_slot[1] * Plan::kSlotBytes;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    if (kPair && stage_w.q0 >= args.Lq) break;     // second CTA of a pair whose rows all lie past Lq
                    tma_store_4d(&tm_o, src_o + hf * Plan::kQHalfBytes, hf * 64, stage_w.h, stage_w.q0, stage_w.b);
                    if (kStageSlots > 1)
                        tma_store_4d(&tm_to, src_t + hf * Plan::kQHalfBytes, hf * 64, stage_w.h, stage_w.q0, stage_w.b);
                }
                tma_store_commit();
                stage_pending = false;
                if (!finish) { stores_in_flight = true; return true; }
                tma_store_wait_read();
                // the slots go back to the ring (their `empty` phase is completed here instead of by an MMA commit)
                for (int s = 0; s < kRingStage; ++s) mbar_arrive(smem_u32(&bar_slot_empty[stage_slot[s]]));
                TRACE(18, stage_it);  // producer: staging slots back in the ring
                return true;
            };
            // hands the staging slots of item number `of_it` to the softmax warps; nothing is loaded into them, so
            // their `full` phase is completed by a plain arrival to keep the ring's parities in step
            auto acquire_stage = [&](int of_it, const Item& of_w) -> bool {
                for (int s = 0; s < kRingStage; ++s) {
                    uint32_t dst, bar;
                    if (!acquire(stage_slot[s], dst, bar)) return false;
                    if (!kPair || lead_cta) mbar_arrive(smem_u32(&bar_slot_full[stage_slot[s]]));
                }
                mbar_arrive(smem_u32(&bar_stage_ready));
                TRACE(9, of_it);      // producer: staging slots handed over
                stage_pending = true;
                stage_it = of_it;
                stage_w = of_w;
                return true;
            };
            // Q, tQ of item number `n` (work item `wi`) into its buffer
            auto load_q = [&](int n, const Item& wi) {
                const uint32_t dq = q_addr(n), dtq = tq_addr(n);
                if (kPair) {
                    const uint32_t qbar = map_to_cta(q_full_bar(n), 0u);
                    if (lead_cta) mbar_arrive_expect_tx(q_full_bar(n), 2 * kQTx);
#pragma unroll
                    for (int hf = 0; hf < kHalves; ++hf) {
                        tma_load_4d_pair(dq + hf * Plan::kQHalfBytes, &tm_q, qbar, hf * 64, wi.h, wi.q0, wi.b);
                        if (kHasTQ) tma_load_4d_pair(dtq + hf * Plan::kQHalfBytes, &tm_tq, qbar, hf * 64, wi.h, wi.q0, wi.b);
                    }
                } else {
                    const uint32_t qbar = q_full_bar(n);
                    mbar_arrive_expect_tx(qbar, kQTx);
#pragma unroll
                    for (int hf = 0; hf < kHalves; ++hf) {
                        tma_load_4d(dq + hf * Plan::kQHalfBytes, &tm_q, qbar, hf * 64, wi.h, wi.q0, wi.b);
                        if (kHasTQ) tma_load_4d(dtq + hf * Plan::kQHalfBytes, &tm_tq, qbar, hf * 64, wi.h, wi.q0, wi.b);
                    }
                }
            };
            Item prev_w{};
            int it = 0;
            Walk wk = walk_init(first_item);
            for (int item = first_item; ok && item < n_items; item += item_stride, ++it, walk_step(wk)) {
                w = item_of(wk);
                const bool has_next = n_items - item > item_stride;
                Walk wk_next = wk;
                walk_step(wk_next);
                if (!kDoubleQ) {
                    // one Q/tQ buffer: it is free once all score MMAs of the item before are complete
                    if (it > 0) ok = mbar_wait(smem_u32(&bar_q_free), (it - 1) & 1, abort_state);
                    if (!ok) break;
                    TRACE(1, it);         // producer: Q, tQ may be replaced
                    load_q(it, w);
                    if (has_next) {
                        // the next item's Q, tQ can only be loaded once this item's score MMAs are done: have them
                        // waiting in L2 by then
                        const Item nx = item_of(wk_next);
#pragma unroll
                        for (int hf = 0; hf < kHalves; ++hf) {
                            tma_prefetch_4d(&tm_q, hf * 64, nx.h, nx.q0, nx.b);
                            if (kHasTQ) tma_prefetch_4d(&tm_tq, hf * 64, nx.h, nx.q0, nx.b);
                        }
                    }
                } else if (it == 0) {
                    load_q(0, w);         // later items: loaded during the item before (below)
                }
                if (!(stream_items && it > 0)) {
                    for (int t = 0; ok && t < kBufs && t < w.n_kv; ++t) ok = load_k(t);
                }
                // staging slots of the item before: after this item's leading K tiles (which the first score MMAs
                // need at once) and before its V tiles (which are not needed until the first softmax is through)
                if (kRingStage > 0 && ok && it > 0) ok = acquire_stage(it - 1, prev_w);
                bool next_q_loaded = false;
                // a leading K tile of the next item (stream_items), in the ring position where the MMA warp consumes it
                auto load_k_of_next = [&](int t) -> bool {
                    const Item cur = w;
                    w = item_of(wk_next);
                    const bool r = load_k(t);
                    w = cur;
                    return r;
                };
                for (int j = 0; ok && j < w.n_kv; ++j) {
                    if (j >= 1) {
                        const int kn = j + kBufs - 1;        // the K tile consumed after V(j - 1)
                        if (kn < w.n_kv) ok = load_k(kn);
                        else if (stream_items && has_next) ok = load_k_of_next(kn - w.n_kv);
                    }
                    if (ok) ok = load_v(j);
                    // the previous item's outputs: the loads above do not depend on its epilogue, the later ones do
                    // (Long enough items with two Q/tQ buffers: the stores go out at j = 1 or 2 if the staged tiles
                    // are complete by then, at j = 3 at the latest; the next item's Q, tQ follow one tile after them.)
                    constexpr bool kTwoStep = kPair && kDoubleQ && kStageSlots > 0;
                    const bool two_step = kTwoStep && w.n_kv >= 6;
                    if (two_step) {
                        if (ok && stores_in_flight) store_staged_finish();          // (issued during the tile before)
                        if (ok && stage_pending && j >= 1) ok = store_staged(j < 3, false);
                    }
                    if (ok && (two_step ? (!stage_pending && !stores_in_flight && j >= 1)
                                        : (j == 1 || j + 1 == w.n_kv))) {
                        if (stage_pending) ok = store_staged();
                        if (kDoubleQ && ok && has_next && !next_q_loaded) {
                            // Two Q/tQ buffers: the other buffer held the item before and then its staged output
                            // tiles, which the stores above have just read (split-KV stages nothing: there the
                            // buffer is free once that item's score MMAs are complete).
                            if (kStageSlots == 0 && it > 0) ok = mbar_wait(smem_u32(&bar_q_free), (it - 1) & 1, abort_state);
                            if (ok) {
                                TRACE(1, it + 1);     // producer: Q, tQ buffer of the next item is free
                                load_q(it + 1, item_of(wk_next));
                                next_q_loaded = true;
                            }
                        }
                    }
                }
                if (ok && stream_items && has_next) ok = load_k_of_next(kBufs - 1);    // consumed after V(n - 1)
                prev_w = w;
                if (kDoubleQ && kStageSlots > 0 && ok) {
                    // this item's output tiles will be staged in its own Q/tQ buffer; stored during the next item
                    stage_pending = true;
                    stage_it = it;
                    stage_w = w;
                }
                // the CTA's last item: its staging slots follow its last V tile
                if (kRingStage > 0 && ok && !has_next) ok = acquire_stage(it, w);
            }
            if (ok && stage_pending) ok = store_staged();
            if (kStageSlots > 0) tma_store_wait_all();
            if (!ok) {
                // Abandoning the work: let the copies already in flight land before the CTA exits.
                // Walk back over the last positions handed out (at most one lap): each slot's current `full`
                // phase completes when its copy has landed (or at once, for a staging slot).
                const int back = r_lapped ? kSlots : r_slot;
                int slot = r_slot;
                uint32_t par = r_parity;
                for (int u = 0; u < back; ++u) {
                    if (slot == 0) { slot = kSlots; par ^= 1u; }
                    --slot;
                    const uint32_t bar = smem_u32(&bar_slot_full[slot]);
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar, par) && globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == kMmaWarp && lead_cta) {
        // =====================================================================================
        // MMA issuer (CTA pair: of the first CTA only, for both).  The whole warp walks the loop in lock step, so that addresses, descriptors and
        // loop state stay warp-uniform; one elected lane issues every tcgen05.mma and the commits
        // that track them.
        // =====================================================================================
        {
            // (CTA pair: M = 256, 128 rows in each CTA; N counts the columns of both CTAs' parts of the B operand)
            constexpr int kMmaM = kPair ? 2 * kBlockM : kBlockM;
            constexpr uint32_t kIdescS1 = make_idesc(kHasTKV ? 2 * kBN : kBN, false, kMmaM);  // Q x [K;tK] or Q x K
            constexpr uint32_t kIdescS2 = make_idesc(kBN, false, kMmaM);                          // tQ x K
            constexpr uint32_t kIdescPV = make_idesc(kHasTKV ? 2 * D : D, true, kMmaM);               // P~ x [V|tV] or P~ x V
            constexpr uint32_t kIdescHV = make_idesc(D, true, kMmaM);                                 // H~ x V
            constexpr uint32_t kVLbo = Plan::kKvHalfBytes;   // bytes between 64-wide N atoms of a V slot
            const bool leader = elect_one();
            bool ok = true;
            uint32_t q_lo = make_desc_lo(q_addr(0), 16);     // set per item (two Q/tQ buffers alternate)
            uint32_t tq_lo = make_desc_lo(tq_addr(0), 16);

            // The hardware queue in front of the tensor pipe is short (about eight instructions), and this
            // warp competes for issue slots with the softmax warps, so whatever runs between two
            // groups of MMAs is kept to a minimum: per key tile there is ONE burst that issues the value MMAs
            // of tile j and the score MMAs of tile j+2, and the barriers the NEXT burst depends on are tested in
            // the middle of it, while the queue is still full.  Only if a test fails does the warp block.
            // Ring position -> (slot, parity) is tracked incrementally.
            struct RingPos { int slot; uint32_t parity; };
            auto advance = [&](RingPos& r) { if (++r.slot == kSlots) { r.slot = 0; r.parity ^= 1u; } };
            auto wait_full = [&](const RingPos& r) -> bool {
                const uint32_t bar = smem_u32(&bar_slot_full[r.slot]);
                if (__all_sync(0xffffffffu, mbar_test_wait(bar, r.parity))) return true;
                return mbar_wait_warp(bar, r.parity, abort_state);
            };

            // Operand descriptors: per operand only the low word of its first k-step is kept in a register (Q and
            // tQ never move; the ring slot's words are set by prepare_*() before the burst that uses them).  The
            // k-steps differ by compile-time constants, so that inside a burst a descriptor costs one add with an
            // immediate and one move beside the tcgen05.mma itself, and the issuing warp stays small in registers.
            uint32_t k_lo = 0, v_lo = 0;
            auto prepare_k = [&](int slot) { k_lo = make_desc_lo(smem_ring + slot * Plan::kSlotBytes, 16); };
            auto prepare_v = [&](int slot) { v_lo = make_desc_lo(smem_ring + slot * Plan::kSlotBytes, kVLbo); };
            auto qd = [&](int k) { return make_desc(q_lo + (((k / 4) * Plan::kQHalfBytes + (k % 4) * 32) >> 4)); };
            auto tqd = [&](int k) { return make_desc(tq_lo + (((k / 4) * Plan::kQHalfBytes + (k % 4) * 32) >> 4)); };
            // B operand of the stacked score MMA: per 64-column half [K (8 KB)][tK (8 KB)]; CTA pair: this CTA's
            // tensor alone, half after half
            // CTA pair without K/V tangents: this CTA's 32 rows of K, halves of 4 KB from the slot's start (see load_k)
            constexpr bool kPairRowsOnly = kPair && !kHasTKV;
            constexpr uint32_t kPairOff2 = kHasTKV ? kHalves * Plan::kKvHalfBytes : 0;   // pair: the slot's second region
            auto kd = [&](int k) {
                return make_desc(k_lo + (((k / 4) * (kPairRowsOnly ? Plan::kKvHalfBytes / 2
                                                     : (kPair ? 1 : Plan::kTilesPerSlot) * Plan::kKvHalfBytes)
                                          + (k % 4) * 32) >> 4));
            };
            // B operand of tQ K^T: the K rows of the same stack; CTA pair: this CTA's 32 rows of K (halves of 4 KB)
            auto k2d = [&](int k) {
                return kPair ? make_desc(k_lo + ((kPairOff2 + (k / 4) * (Plan::kKvHalfBytes / 2) + (k % 4) * 32) >> 4)) : kd(k);
            };
            auto vd = [&](int k) { return make_desc(v_lo + k * (2048 >> 4)); };
            // B operand of H~ V: the V atoms of the same slot; CTA pair: this CTA's one atom of V
            auto v2d = [&](int k) { return kPair ? make_desc(v_lo + ((kPairOff2 + k * 2048) >> 4)) : vd(k); };
            // issue and completion tracking in the form the kernel variant needs
            const uint32_t lead_pred = leader ? 1u : 0u;     // all lanes run the issue code, this lane's instructions take effect
            auto mma_ss0 = [&](uint32_t d, uint64_t a, uint64_t b, uint32_t idesc) { mma_ss_if<false, kPair>(lead_pred, d, a, b, idesc); };
            auto mma_ss1 = [&](uint32_t d, uint64_t a, uint64_t b, uint32_t idesc) { mma_ss_if<true, kPair>(lead_pred, d, a, b, idesc); };
            auto mma_tsx = [&](uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
                mma_ts_if<kPair>(lead_pred, d, a, b, idesc, acc);
            };
            auto commit = [&](uint32_t bar) { tc_commit_if<kPair>(lead_pred, bar); };

            // score MMAs of global tile g (issued by the elected lane), in two parts so that the look-ahead for
            // the next tile can run between them; `last_of_item`: these are the item's last score MMAs
            auto issue_scores_a = [&](int g, int buf) {
                const uint32_t tm_s = tmem + kScoreCol0 + buf * kScoreBufStride;
                if (leader) TRACE(21, g);         // MMA: about to issue score MMAs
                mma_ss0(tm_s, qd(0), kd(0), kIdescS1);
#pragma unroll
                for (int k = 1; k < D / 16; ++k) mma_ss1(tm_s, qd(k), kd(k), kIdescS1);
            };
            auto issue_scores_b = [&](int g, int buf, int slot, bool last_of_item) {
                const uint32_t tm_ts = tmem + kScoreCol0 + buf * kScoreBufStride + kBN;
                if (kHasTQ) {
                    if (kHasTKV) mma_ss1(tm_ts, tqd(0), k2d(0), kIdescS2);
                    else mma_ss0(tm_ts, tqd(0), k2d(0), kIdescS2);
#pragma unroll
                    for (int k = 1; k < D / 16; ++k) mma_ss1(tm_ts, tqd(k), k2d(k), kIdescS2);
                }
                commit(smem_u32(&bar_slot_empty[slot]));
                commit(smem_u32(&bar_s_full[buf]));
                if (last_of_item) commit(smem_u32(&bar_q_free));
                if (leader) TRACE(2, g);          // MMA: score MMAs of tile g issued
            };
            // value MMAs of tile j of the item (global tile g) out of ring slot `slot`: those that read P~, then
            // those that read H~
            auto issue_values_p = [&](int j, int g, int buf) {
                const uint32_t tm_p = tmem + kScoreCol0 + buf * kScoreBufStride;
                if (leader) TRACE(3, g);          // MMA: about to issue value MMAs
#pragma unroll
                for (int k = 0; k < kBN / 16; ++k) {
                    mma_tsx(tmem_o, tm_p + k * 8, vd(k), kIdescPV, (j > 0 || k > 0) ? 1u : 0u);
                }
            };
            auto issue_values_h = [&](int j, int g, int buf, int slot) {
                const uint32_t tm_h = tmem + kScoreCol0 + buf * kScoreBufStride + kBN;
                if (kHasTQ) {
#pragma unroll
                    for (int k = 0; k < kBN / 16; ++k) {
                        mma_tsx(tmem_t, tm_h + k * 8, v2d(k), kIdescHV, (kHasTKV || j > 0 || k > 0) ? 1u : 0u);
                    }
                }
                commit(smem_u32(&bar_slot_empty[slot]));
                commit(smem_u32(&bar_pv_done[g & 1]));
                if (leader) TRACE(4, g);          // MMA: value MMAs of tile g issued
            };
            // what the burst of global tile g needs: V and K(+2) in shared memory, P~/H~ in tensor memory
            // The three tests are issued back to back (their latencies overlap) and agreed on with one vote:
            // bit 0 = the V and K slots are full, bit 1 = P~ (and H~) are in tensor memory.
            auto test_tile = [&](const RingPos& pv, const RingPos& pk, bool has_k, const BufPos& bp) -> uint32_t {
                const bool tv = mbar_test_wait(smem_u32(&bar_slot_full[pv.slot]), pv.parity);
                const bool tk = mbar_test_wait(smem_u32(&bar_slot_full[has_k ? pk.slot : pv.slot]), has_k ? pk.parity : pv.parity);
                const bool tp = mbar_test_wait(smem_u32(&bar_p_full[bp.buf]), bp.phase);
                if (__all_sync(0xffffffffu, tv & tk & tp)) return 3u;
                return __all_sync(0xffffffffu, tv & tk) ? 1u : 0u;
            };
            // blocks for whatever test_tile() did not see (`seen`: its result)
            auto wait_tile = [&](const RingPos& pv, const RingPos& pk, bool has_k, int g, const BufPos& bp, uint32_t seen) -> bool {
                if (leader) TRACE(22, g);   // MMA: has to block for tile g
                bool r = true;
                if (!(seen & 1u)) {
                    r = wait_full(pv);
                    if (r && has_k) r = wait_full(pk);
                    if (leader) TRACE(19, g);   // MMA: the tile's V and K slots are full
                }
                if (r && !(seen & 2u)) r = mbar_wait_warp(smem_u32(&bar_p_full[bp.buf]), bp.phase, abort_state);
                return r;
            };

            // Ring order (as the producer fills it), per item: K0, K1, V0, K2, V1, K3, ...
            ACC_DECL(acc_mma_tile);     // blocked for a tile's barriers inside an item
            ACC_DECL(acc_mma_item);     // blocked at an item's start (first V and K tiles, first P~, accumulators free)
            RingPos pos{0, 0u};
            BufPos bp{0, 0u};    // score buffer / phase of the tile whose value MMAs come next
            int g0 = 0;          // global number of the item's first key tile
            int it = 0;
            Walk wk = walk_init(first_item);
            for (int item = first_item; ok && item < n_items; item += item_stride, ++it, walk_step(wk)) {
                const Item w = item_of(wk);
                const int n_kv = w.n_kv;
                const bool has_next_item = n_items - item > item_stride;
                // stream_items: this item's leading score MMAs went out with the last bursts of the item before
                const bool leading_done = stream_items && it > 0;
                // ... and the next item's go out with the last bursts of this one
                const bool feeds_next = stream_items && has_next_item;
                ok = mbar_wait_warp(q_full_bar(it), q_full_phase(it), abort_state);
                if (leader) TRACE(10, it);    // MMA: Q, tQ of the item seen
                q_lo = make_desc_lo(q_addr(it), 16);
                tq_lo = make_desc_lo(tq_addr(it), 16);
                // the item's leading score MMAs: one tile per score buffer
                for (int t = leading_done ? kBufs : 0; ok && t < kBufs && t < n_kv; ++t) {
                    ok = wait_full(pos);
                    if (!ok) break;
                    if (t == 0) {
                        if (leader) TRACE(11, it);    // MMA: K(0) of the item seen
                        tc_fence_after();
                    }
                    prepare_k(pos.slot);
                    // (leading tile t sits t score buffers after the item's first tile: t < kBufs, no phase needed)
                    const int lbuf = bp.buf + t < kBufs ? bp.buf + t : bp.buf + t - kBufs;
                    issue_scores_a(g0 + t, lbuf);
                    issue_scores_b(g0 + t, lbuf, pos.slot, t + 1 == n_kv);
                    advance(pos);
                }
                if (!ok) break;
                // the ring positions between the item's leading K tiles and V(0) stage the previous item's outputs
                if (it > 0) { for (int s = 0; s < kRingStage; ++s) advance(pos); }
                // pos = V(0).  Per tile j: burst = value MMAs of tile j, score MMAs of tile j + kBufs; the barriers of
                // tile j+1 are tested in the middle of the burst, while the queue is still full.
                RingPos pos_v = pos, pos_k = pos;
                bool has_k = n_kv > kBufs || feeds_next;      // (stream_items implies n_kv >= kBufs)
                advance(pos);
                pos_k = pos;
                if (has_k) advance(pos);
                ACC_BEGIN(acc_mma_item);
                ok = wait_tile(pos_v, pos_k, has_k, g0, bp, 0u);
                // the first value MMA of an item overwrites O and T: the previous item's epilogue must have read them
                if (ok && it > 0) ok = mbar_wait_warp(smem_u32(&bar_acc_free), (it - 1) & 1, abort_state);
                ACC_END(acc_mma_item);
                if (!ok) break;
                prepare_v(pos_v.slot);
                if (has_k) prepare_k(pos_k.slot);
                for (int j = 0; ok && j < n_kv; ++j) {
                    if (feeds_next && j + kBufs == n_kv) {
                        // from here on the score MMAs are those of the next item's leading tiles: its Q, tQ (loaded
                        // during this item into the other buffer)
                        ok = mbar_wait_warp(q_full_bar(it + 1), q_full_phase(it + 1), abort_state);
                        if (!ok) break;
                        q_lo = make_desc_lo(q_addr(it + 1), 16);
                        tq_lo = make_desc_lo(tq_addr(it + 1), 16);
                    }
                    if (leader) TRACE(29, g0 + j);   // MMA: burst of tile j begins (loop top)
                    tc_fence_after();
                    if (leader) TRACE(30, g0 + j);   // MMA: after the tensor-core fence
                    issue_values_p(j, g0 + j, bp.buf);
                    issue_values_h(j, g0 + j, bp.buf, pos_v.slot);
                    if (has_k) issue_scores_a(g0 + j + kBufs, bp.buf);    // tile j + kBufs reuses tile j's buffer
                    // Middle of the burst, the queue in front of the tensor pipe is full: everything the next burst
                    // needs is worked out here (its ring positions, score buffer, operand descriptors, and a test
                    // of its barriers), so that after the last score MMA only the commits stand between this
                    // burst and the next one.
                    const bool nxt_exists = j + 1 < n_kv;
                    const bool nxt_has_k = j + 1 + kBufs < n_kv || feeds_next;
                    const RingPos nxt_v = pos;
                    RingPos nxt_k = pos;
                    BufPos bp_next = bp;
                    next_buf(bp_next);
                    uint32_t nxt_seen = 3u;
                    uint32_t v_lo_next = v_lo, k_lo_next = k_lo;
                    if (nxt_exists) {
                        advance(pos);
                        nxt_k = pos;
                        if (nxt_has_k) advance(pos);
                        nxt_seen = test_tile(nxt_v, nxt_k, nxt_has_k, bp_next);
                        v_lo_next = make_desc_lo(smem_ring + nxt_v.slot * Plan::kSlotBytes, kVLbo);
                        if (nxt_has_k) k_lo_next = make_desc_lo(smem_ring + nxt_k.slot * Plan::kSlotBytes, 16);
                    }
                    // (tile j + kBufs of this item, or tile j + kBufs - n_kv of the next one: either way its last tile
                    // has index n_kv - 1 there, all items being equally long in stream_items)
                    if (has_k) issue_scores_b(g0 + j + kBufs, bp.buf, pos_k.slot, j + kBufs + 1 == n_kv || j + kBufs + 1 == 2 * n_kv);
                    if (leader) TRACE(23, g0 + j);   // MMA: burst of tile j issued
                    if (nxt_seen != 3u) {
                        ACC_BEGIN(acc_mma_tile);
                        ok = wait_tile(nxt_v, nxt_k, nxt_has_k, g0 + j + 1, bp_next, nxt_seen);
                        ACC_END(acc_mma_tile);
                    }
                    v_lo = v_lo_next;
                    k_lo = k_lo_next;
                    bp = bp_next;
                    pos_v = nxt_v;
                    pos_k = nxt_k;
                    has_k = nxt_has_k;
                }
                g0 += n_kv;
            }
            ACC_WRITE(0, acc_mma_tile);
            ACC_WRITE(1, acc_mma_item);
            if (!ok && leader) {
                // Abandoning the work: wait (bounded) until the tensor core has drained what was issued.
                commit(smem_u32(&bar_drain));
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(smem_u32(&bar_drain), 0) && globaltimer_ns() - t0 < 100000000ull) {}
            }
            __syncwarp();
        }
    }
    } else {
        if (kMoveRegs) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmaxWarps));
        // =====================================================================================
        // Softmax warps.  Thread (warp w, lane) owns query row 32*(w%4) + lane (= its tensor-memory
        // lane) and all columns of every score tile.
        //
        // With two groups, group (g & 1) takes key tile g (numbered over all items of the CTA, like the score
        // buffers), so that two tiles are in work at a time and each scheduler has two softmax warps to hide
        // latencies with.  What Algorithm 2 carries from tile to tile is shared as follows.  The reference max m
        // (and, once per item, the centring constant of tS) goes through shared memory in tile order: the group
        // of tile g waits for the decision of tile g - 1, takes its own, publishes it and only then computes its
        // exponentials, so the groups run half a tile apart.  l and r are summed per group (both relative to the
        // common m); the group of the item's last tile finishes the item: it adds the other group's sums and runs
        // the epilogue while the other group is already in the next item.
        // =====================================================================================
        const int grp = (kGroups == 2) ? ((warp - kFirstSoftmaxWarp) >> 2) : 0;
        // one group: warps 4..7 of this branch are the epilogue warps (same rows, i.e. tensor-memory lanes, as the
        // softmax warp of their quarter)
        constexpr bool kEpiWarps = (kGroups == 1);
        const bool epi_role = kEpiWarps && (warp - kFirstSoftmaxWarp) >= 4;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                          // 0..127: a warp may only touch lanes 32*(warp%4)..+31
        const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
        const float c1 = args.scale_log2;
        const float sc = args.scale;
        const bool neg_scale = c1 < 0.0f;
        bool ok = true;
        int g0 = 0;          // global number of the item's first key tile
        BufPos bp{0, 0u};    // score buffer / phase of tile g0 + j, advanced for every tile (also the other group's)
        int it = 0;
        int ring_slot = 0;   // ring slot of the item's first position (the ring hands out 2 n + kStageSlots per item)
        // exchange area of the two groups, one fp32 per row each
        const uint32_t xch_m = smem_base + Plan::kOperandBytes + row * 4;       // reference max after the latest tile
        const uint32_t xch_shift = xch_m + kBlockM * 4;                         // centring constant of the item
        const uint32_t xch_l = xch_m + 2 * kBlockM * 4;                         // partial l of the non-finishing group
        const uint32_t xch_r = xch_m + 3 * kBlockM * 4;                         // partial r
        const uint32_t mbar = smem_u32(&bar_m[quarter]);
        const uint32_t finbar = smem_u32(&bar_fin[quarter]);
        // arrival on a barrier the MMA-issuing warp waits on: CTA pair -> the first CTA's copy of it
        auto arrive_at_issuer = [&](uint32_t bar) {
            if (kPair && !lead_cta) mbar_arrive_cluster(map_to_cta(bar, 0u));
            else mbar_arrive(bar);
        };

        ACC_DECL(acc_sm_scores);   // blocked for a tile's scores
        ACC_DECL(acc_sm_values);   // blocked for the item's last value MMAs (epilogue)
        ACC_DECL(acc_sm_epi);      // epilogue after that wait
        Walk wk = walk_init(first_item);
        for (int item = first_item; ok && item < n_items; item += item_stride, ++it, walk_step(wk)) {
            const Item w = item_of(wk);
            const int n_kv = w.n_kv;
            float m_ref = -INFINITY;   // running reference max, log2 domain (m of Algorithm 2, lazily updated)
            float l_run = 0.0f;        // l (two groups: this group's share)
            float r_run = 0.0f;        // r (of the centred tS, see below; two groups: this group's share)
            float ts_shift = 0.0f;     // per-row constant subtracted from tS
            float m_other = -INFINITY; // two groups: the reference the other group's sums were last known to use
            // two groups: the group of the item's last tile finishes the item
            const bool finisher = (kGroups == 1) || (((g0 + n_kv - 1) & 1) == grp);

            for (int j = 0; j < (epi_role ? 0 : n_kv); ++j) {
                const int g = g0 + j;
                const int bsel = bp.buf;
                const uint32_t bphase = bp.phase;
                next_buf(bp);
                if (kGroups == 2 && (g & 1) != grp) continue;
                ACC_BEGIN(acc_sm_scores);
                if (!mbar_wait_warp(smem_u32(&bar_s_full[bsel]), bphase, abort_state)) { ok = false; break; }
                ACC_END(acc_sm_scores);
                tc_fence_after();
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                const bool trace_me = trace_on && lane == 0;
                if (trace_me && g < kTraceSteps) g_trace[5 + ((warp - kFirstSoftmaxWarp) & 3)][g] = clock64();     // softmax warp: scores seen ready
#endif
                const uint32_t tm_s = tmem + lane_base + kScoreCol0 + bsel * kScoreBufStride;
                const uint32_t tm_ts = tm_s + kBN;

                uint32_t sv[kBN];
                uint32_t tv[kBN];
                // S first; tS is fetched while the row maximum is formed
#pragma unroll
                for (int c0 = 0; c0 < kBN; c0 += 32) TMEM_LD32(tm_s + c0, sv, c0);
                if (kGroups == 1 || !kHasTQ) tc_wait_ld();
                if (kHasTQ) {
#pragma unroll
                    for (int c0 = 0; c0 < kBN; c0 += 32) TMEM_LD32(tm_ts + c0, tv, c0);
                }
                if (kGroups == 2 && kHasTQ) tc_wait_ld();      // (two groups hide the latency by themselves: one wait)
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && quarter == 0 && g < kTraceSteps) g_trace[26][g] = clock64();    // softmax: scores in registers
#endif

                // keys past Lk (zero-filled by TMA) must not enter the softmax
                const int valid = args.Lk - (w.tile0 + j) * kBN;
                if (valid < kBN) {
                    const uint32_t masked = neg_scale ? 0x7F800000u : 0xFF800000u;   // -inf after scaling
#pragma unroll
                    for (int c = 0; c < kBN; ++c) if (c >= valid) sv[c] = masked;
                }

                // rowmax(S_ij) (four independent chains), in the log2 domain
                float mx4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) mx4[u] = __uint_as_float(sv[u]);
                if (!neg_scale) {
#pragma unroll
                    for (int c = 4; c < kBN; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(sv[c]));
                } else {
#pragma unroll
                    for (int c = 4; c < kBN; ++c) mx4[c & 3] = fminf(mx4[c & 3], __uint_as_float(sv[c]));
                }
                float mx = neg_scale ? fminf(fminf(mx4[0], mx4[1]), fminf(mx4[2], mx4[3]))
                                     : fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                mx *= c1;

                if (kGroups == 2) {
                    // The decision of tile g - 1 (the other group's) comes first, also across items: the exchange
                    // words are single and are written strictly in tile order.
                    if (g > 0 && !mbar_wait_warp(mbar, (g - 1) & 1, abort_state)) { ok = false; break; }
                    if (j > 0) {
                        const float m_prev = ld_shared_f32(xch_m);
                        if (j == 1) ts_shift = ld_shared_f32(xch_shift);
                        m_other = m_prev;
                        if (m_prev > m_ref) {
                            // this group's sums move to the common reference (0 * 0 on its first tile)
                            const float f = ex2f(m_ref - m_prev);
                            l_run *= f;
                            r_run *= f;
                            m_ref = m_prev;
                        }
                    }
                }
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && quarter == 0 && g < kTraceSteps) g_trace[27][g] = clock64();    // softmax: reference of tile g-1 seen
#endif
                // tO does not change when a per-row constant is subtracted from tS (softmax is shift invariant:
                // the constant leaves H~ V - (r/l) O unchanged).  Centring tS on its mean over the item's first
                // tile keeps H~ and r small, so that the bf16 rounding of H~ scales with |tS - mu| instead of |tS|
                // when the two terms cancel in the epilogue.  (Keys past Lk are zero-filled, so their tS is exactly
                // 0 and they drop out of the sum.)
                auto centre_of_first_tile = [&]() {
                    float sm4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                    for (int c = 0; c < kBN; ++c) sm4[c & 3] += __uint_as_float(tv[c]);
                    const int n_valid = valid < kBN ? valid : kBN;
                    return sc * ((sm4[0] + sm4[1]) + (sm4[2] + sm4[3])) / static_cast<float>(n_valid);
                };
                if (kHasTQ && kGroups == 1) tc_wait_ld();      // tS is in registers
                if (kHasTQ && j == 0) ts_shift = centre_of_first_tile();

                // m_new = max(m, rowmax), applied lazily: the result does not depend on which
                // reference is used as long as exp() stays in range.
                const bool need = mx > m_ref + kRescaleThreshold;
                const float alpha = need ? ex2f(m_ref - mx) : 1.0f;    // e^{m - m_new}; 0 on the first tile (m = -inf)
                m_ref = need ? mx : m_ref;
                // (whether any row of the warp rescales: asked here, acted on after the pass over the columns, so that
                // the vote's latency and the branch stay off the path to the first exponential)
                const bool any_need = j > 0 && __any_sync(0xffffffffu, need);
                // Rescale of the accumulators where the reference moved (rare: once or twice per row).  One softmax
                // group: after the pass over the columns (the branch and the vote's latency stay off the path to the
                // first exponential); two groups with tangents: before it (their register budget is tighter, and the packed P~, H~
                // would have to live across the branch).
                auto rescale_accumulators = [&]() -> bool {
                    // the accumulators must be complete up to tile j-1 before they are rescaled
                    if (!mbar_wait_warp(smem_u32(&bar_pv_done[(g - 1) & 1]), ((g - 1) >> 1) & 1, abort_state)) return false;
                    tc_fence_after();
                    constexpr int kAccCols = kHasTQ ? 2 * D : D;
#pragma unroll 1
                    for (int c0 = 0; c0 < kAccCols; c0 += 32) {
                        uint32_t acc[32];
                        TMEM_LD32(tmem_o + lane_base + c0, acc, 0);
                        tc_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) acc[c] = __float_as_uint(__uint_as_float(acc[c]) * alpha);
                        TMEM_ST32(tmem_o + lane_base + c0, acc, 0);
                    }
                    return true;
                };
                constexpr bool kLateRescale = (kGroups == 1) || !kHasTQ;
                if (!kLateRescale && any_need && !rescale_accumulators()) { ok = false; break; }
                l_run *= alpha;
                r_run *= alpha;
                if (kGroups == 2) {
                    // publish the decision (and the item's centring constant): the other group may go on
                    st_shared_f32(xch_m, m_ref);
                    if (j == 0) st_shared_f32(xch_shift, ts_shift);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(mbar);
                }

                // P~ = exp(S - m_new), l += rowsum(P~), H~ = P~ . tS, r += rowsum(H~), and both rounded to bf16, in ONE
                // pass over the columns (two columns per FMA-pipe instruction).  The exponentials set the pace of the
                // pass (the special-function unit takes 8 cycles per warp instruction, 64 of them per tile), and
                // everything else fits into the issue slots they leave free; as separate passes the H~ arithmetic
                // and the conversions came on top.
                const uint64_t c1c1 = pack_f32x2(c1, c1);
                const uint64_t negm = pack_f32x2(-m_ref, -m_ref);
                const uint64_t scsc = pack_f32x2(sc, sc);
                const uint64_t negshift = pack_f32x2(-ts_shift, -ts_shift);
                uint32_t pk_p[kBN / 2];
                uint32_t pk_h[kBN / 2];
                float lsum, rsum = 0.0f;
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && quarter == 0 && g < kTraceSteps) g_trace[24][g] = clock64();    // softmax: the pass over the columns begins
#endif
                // (Keys past Lk of the item's ragged last tile: their S was set to -inf after scaling above, so P~ is
                // exactly 0 whatever the scale, the host having replaced a zero scale by 2^-100; their tS is exactly
                // 0, hence H~ = 0 * (-shift) = 0.)
                {
                    uint64_t ls2[2] = {0ull, 0ull};     // (+0.0f, +0.0f)
                    uint64_t rs2[2] = {0ull, 0ull};
#pragma unroll
                    for (int c = 0; c < kBN; c += 2) {
                        float x0, x1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), c1c1, negm), x0, x1);
                        const float p0 = ex2f(x0), p1 = ex2f(x1);
                        const uint64_t p2 = pack_f32x2(p0, p1);
                        ls2[(c >> 1) & 1] = add_f32x2(ls2[(c >> 1) & 1], p2);
                        pk_p[c >> 1] = pack_bf16(p0, p1);
                        if (kHasTQ) {
                            const uint64_t ts2 = fma_f32x2(pack_f32x2(__uint_as_float(tv[c]), __uint_as_float(tv[c + 1])), scsc, negshift);
                            const uint64_t h2 = mul_f32x2(p2, ts2);
                            float h0, h1;
                            unpack_f32x2(h2, h0, h1);
                            rs2[(c >> 1) & 1] = add_f32x2(rs2[(c >> 1) & 1], h2);
                            pk_h[c >> 1] = pack_bf16(h0, h1);
                        }
                    }
                    float a0, a1, a2, a3;
                    unpack_f32x2(ls2[0], a0, a1);
                    unpack_f32x2(ls2[1], a2, a3);
                    lsum = (a0 + a1) + (a2 + a3);
                    if (kHasTQ) {
                        unpack_f32x2(rs2[0], a0, a1);
                        unpack_f32x2(rs2[1], a2, a3);
                        rsum = (a0 + a1) + (a2 + a3);
                    }
                }
                l_run += lsum;
                r_run += rsum;
                if (kLateRescale && any_need && !rescale_accumulators()) { ok = false; break; }
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && quarter == 0 && g < kTraceSteps) g_trace[25][g] = clock64();    // softmax: ... and ends
#endif
#pragma unroll
                for (int c0 = 0; c0 < kBN / 2; c0 += 32) TMEM_ST32(tm_s + c0, pk_p, c0);      // bf16: two keys per column
                if (kHasTQ) TMEM_ST32(tm_ts, pk_h, 0);
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && quarter == 0 && g < kTraceSteps) g_trace[28][g] = clock64();    // softmax: P~, H~ stores issued
#endif
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_at_issuer(smem_u32(&bar_p_full[bsel]));
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
                if (trace_me && g < kTraceSteps) g_trace[13 + ((warp - kFirstSoftmaxWarp) & 3)][g] = clock64();    // softmax warp: arrived
#endif
            }
            if (!ok) break;

            // Ring positions of this item: 2 n_kv tiles, plus the previous item's staging slots.  Its own staging
            // slots come after the next item's leading K tiles (every item has n_kv tiles here: the kernel that
            // cuts the keys into chunks stages nothing), or right after its last V tile if it is the CTA's last.
            int stage_slot_o = 0;
            if (kRingStage > 0) {
                const bool has_next = n_items - item > item_stride;
                const int next_start = (ring_slot + 2 * (n_kv % kSlots) + (it > 0 ? kRingStage : 0)) % kSlots;
                stage_slot_o = has_next ? (next_start + min(kBufs, n_kv)) % kSlots : next_start;
                ring_slot = next_start;
            }

            if (kGroups == 2 && !finisher) {
                // This group's share of l and r goes to the group that finishes the item; the exchange words are
                // single, so the finisher of the item before must have read its own first.
                if (it > 0 && !mbar_wait_warp(smem_u32(&bar_fin_read[quarter]), (it - 1) & 1, abort_state)) { ok = false; break; }
                st_shared_f32(xch_l, l_run);
                st_shared_f32(xch_r, r_run);
                __syncwarp();
                if (lane == 0) mbar_arrive(finbar);
                g0 += n_kv;
                continue;
            }

            if (kEpiWarps) {
                // One group: l, r, m and the centring constant of the finished item go to the epilogue warp of this
                // quarter of the rows through the exchange words (single: the epilogue warp must have read the item
                // before's), and the softmax warp goes on to the next item at once.
                if (!epi_role) {
                    if (it > 0 && !mbar_wait_warp(smem_u32(&bar_fin_read[quarter]), (it - 1) & 1, abort_state)) { ok = false; break; }
                    st_shared_f32(xch_l, l_run);
                    st_shared_f32(xch_r, r_run);
                    st_shared_f32(xch_m, m_ref);
                    st_shared_f32(xch_shift, ts_shift);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(finbar);
                    g0 += n_kv;
                    continue;
                }
                if (!mbar_wait_warp(finbar, it & 1, abort_state)) { ok = false; break; }
                l_run = ld_shared_f32(xch_l);
                r_run = ld_shared_f32(xch_r);
                m_ref = ld_shared_f32(xch_m);
                ts_shift = ld_shared_f32(xch_shift);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_fin_read[quarter]));
            }

            // Epilogue: O/l, L = m + log l, tO = (T - r (O/l)) / l, once the item's last value MMAs are complete
            // (which implies all earlier ones).  A parity wait on bar_pv_done[g & 1] for tile g means what it should
            // only once the value MMAs of tile g - 2 (the barrier's previous phase) are known to be complete.  The
            // scores of tile g_last have been seen, and their completion implies that of everything issued before
            // them: the value MMAs up to tile g_last - kBufs, and for an item's leading tiles those of all earlier
            // items.  That covers g_last - 3, so tile g_last - 1 can be waited for first, and g_last after it.
            const int g_last = g0 + n_kv - 1;
            ACC_BEGIN(acc_sm_values);
            if (n_kv >= 2) ok = mbar_wait_warp(smem_u32(&bar_pv_done[(g_last - 1) & 1]), ((g_last - 1) >> 1) & 1, abort_state);
            if (ok) ok = mbar_wait_warp(smem_u32(&bar_pv_done[g_last & 1]), (g_last >> 1) & 1, abort_state);
            if (ok && kGroups == 2) {
                // the other group's sums, brought to the final reference (it last knew m_other; 0 if it had no tile)
                ok = mbar_wait_warp(finbar, it & 1, abort_state);
                if (ok) {
                    const float f = ex2f(m_other - m_ref);
                    l_run = fmaf(ld_shared_f32(xch_l), f, l_run);
                    r_run = fmaf(ld_shared_f32(xch_r), f, r_run);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_fin_read[quarter]));
                }
            }
            ACC_END(acc_sm_values);
            ACC_BEGIN(acc_sm_epi);
            if (!ok) break;
            tc_fence_after();
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
            if (trace_on && lane == 0 && ((warp - kFirstSoftmaxWarp) & 3) == 0 && it < kTraceSteps) g_trace[12][it] = clock64();    // softmax warp: epilogue begins
#endif
            const float l_tot = l_run, r_tot = r_run;
            const int qi = w.q0 + row;
            const bool in_range = qi < args.Lq;
            const float inv_l = 1.0f / l_tot;
            const float mu = r_tot * inv_l;
            const int b = w.b, h = w.h, split = w.split;
            const size_t row_off = ((static_cast<size_t>(b) * args.Lq + (in_range ? qi : 0)) * args.H + h) * D;
            // split-KV: this chunk's normalised partial results go to the fp32 scratch of chunk `split`
            const size_t part_off = kSplit ? static_cast<size_t>(split) * args.B * args.Lq * args.H * D + row_off : 0;
            float* po_row = kSplit ? args.part_o + part_off : nullptr;
            float* pto_row = (kSplit && kHasTQ) ? args.part_to + part_off : nullptr;
            // bf16 outputs: staged in the ring slots after the item's last V tile, in the 128-byte-swizzled
            // layout of the output tensor maps (row r, 16-byte chunk c of a 64-column half at r*128 + (c ^ (r&7))*16)
            uint32_t stage_o = 0, stage_t = 0;
            if (kRingStage > 0) {
                stage_o = smem_ring + stage_slot_o * Plan::kSlotBytes + row * 128;
                stage_t = smem_ring + ((stage_slot_o + 1) % kSlots) * Plan::kSlotBytes + row * 128;
            } else if (kStageSlots > 0) {
                // two Q/tQ buffers: the item's own Q and tQ tiles are dead (its last value MMAs are complete, hence
                // every MMA issued before them) and have the size and layout of its output tiles
                stage_o = q_addr(it) + row * 128;
                stage_t = tq_addr(it) + row * 128;
            }
            if (kSplit || !kEpiWarps) {
                // (two softmax groups: the epilogue shares its registers with the softmax pass, so it stays a rolled
                // loop over 32-column chunks that stages each chunk at once)
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t ov[32];
                    uint32_t tvv[32];
                    TMEM_LD32(tmem_o + lane_base + c0, ov, 0);
                    if (kHasTQ) TMEM_LD32(tmem_t + lane_base + c0, tvv, 0);
                    if (!kSplit && kRingStage > 0 && c0 == 0) {
                        ok = mbar_wait_warp(smem_u32(&bar_stage_ready), it & 1, abort_state);
                        if (!ok) { tc_wait_ld(); break; }
                    }
                    tc_wait_ld();
                    if (c0 + 32 >= D) {
                        // O and T are in registers: the next item's first value MMA may overwrite them
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) arrive_at_issuer(smem_u32(&bar_acc_free));
                    }
                    if (kSplit) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            const float o0 = __uint_as_float(ov[c]) * inv_l;
                            ov[c] = __float_as_uint(o0);
                            if (kHasTQ) tvv[c] = __float_as_uint(fmaf(-mu, o0, __uint_as_float(tvv[c]) * inv_l));
                        }
                        if (in_range) {
#pragma unroll
                            for (int v4 = 0; v4 < 8; ++v4) {
                                *reinterpret_cast<uint4*>(po_row + c0 + v4 * 4) = make_uint4(ov[4 * v4], ov[4 * v4 + 1], ov[4 * v4 + 2], ov[4 * v4 + 3]);
                                if (kHasTQ)
                                    *reinterpret_cast<uint4*>(pto_row + c0 + v4 * 4) = make_uint4(tvv[4 * v4], tvv[4 * v4 + 1], tvv[4 * v4 + 2], tvv[4 * v4 + 3]);
                            }
                        }
                    } else {
                        uint32_t po[16], pt[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float o0 = __uint_as_float(ov[2 * c]) * inv_l;
                            const float o1 = __uint_as_float(ov[2 * c + 1]) * inv_l;
                            po[c] = pack_bf16(o0, o1);
                            if (kHasTQ) {
                                const float t0 = fmaf(-mu, o0, __uint_as_float(tvv[2 * c]) * inv_l);
                                const float t1 = fmaf(-mu, o1, __uint_as_float(tvv[2 * c + 1]) * inv_l);
                                pt[c] = pack_bf16(t0, t1);
                            }
                        }
                        // rows beyond Lq are staged too (the store clips them)
                        const uint32_t half_off = (c0 >> 6) * Plan::kQHalfBytes;
                        const int chunk0 = (c0 & 63) >> 3;
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            const uint32_t off = half_off + (((chunk0 + v4) ^ (row & 7)) << 4);
                            st_shared_v4(stage_o + off, po[4 * v4], po[4 * v4 + 1], po[4 * v4 + 2], po[4 * v4 + 3]);
                            if (kHasTQ) st_shared_v4(stage_t + off, pt[4 * v4], pt[4 * v4 + 1], pt[4 * v4 + 2], pt[4 * v4 + 3]);
                        }
                    }
                }
            } else {
                // The next item's first value MMAs wait for this: first everything that needs the accumulators (32
                // columns of O and T at a time: load, normalise, round to bf16 and keep the packed row in registers),
                // then the accumulators are given back, and only then is the row written to the staging buffer.
                uint32_t po[D / 2];
                uint32_t pt[kHasTQ ? D / 2 : 1];
                const uint64_t inv2 = pack_f32x2(inv_l, inv_l);
                const uint64_t negmu2 = pack_f32x2(-mu, -mu);
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t ov[32];
                    uint32_t tvv[32];
                    TMEM_LD32(tmem_o + lane_base + c0, ov, 0);
                    if (kHasTQ) TMEM_LD32(tmem_t + lane_base + c0, tvv, 0);
                    tc_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const uint64_t o2 = mul_f32x2(pack_f32x2(__uint_as_float(ov[2 * c]), __uint_as_float(ov[2 * c + 1])), inv2);
                        float o0, o1;
                        unpack_f32x2(o2, o0, o1);
                        po[(c0 >> 1) + c] = pack_bf16(o0, o1);
                        if (kHasTQ) {
                            const uint64_t tt = mul_f32x2(pack_f32x2(__uint_as_float(tvv[2 * c]), __uint_as_float(tvv[2 * c + 1])), inv2);
                            float t0, t1;
                            unpack_f32x2(fma_f32x2(negmu2, o2, tt), t0, t1);
                            pt[(c0 >> 1) + c] = pack_bf16(t0, t1);
                        }
                    }
                }
                // O and T are in registers: the next item's first value MMA may overwrite them
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_at_issuer(smem_u32(&bar_acc_free));
                if (kRingStage > 0) {
                    ok = mbar_wait_warp(smem_u32(&bar_stage_ready), it & 1, abort_state);
                    if (!ok) break;
                }
                // rows beyond Lq are staged too (the store clips them)
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    const uint32_t half_off = (c0 >> 6) * Plan::kQHalfBytes;
                    const int chunk0 = (c0 & 63) >> 3;
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        const uint32_t off = half_off + (((chunk0 + v4) ^ (row & 7)) << 4);
                        const int q = (c0 >> 1) + 4 * v4;
                        st_shared_v4(stage_o + off, po[q], po[q + 1], po[q + 2], po[q + 3]);
                        if (kHasTQ) st_shared_v4(stage_t + off, pt[q], pt[q + 1], pt[q + 2], pt[q + 3]);
                    }
                }
            }
            if (!ok) break;
            if (kStageSlots > 0) {
                // the staged tiles are complete: the producer thread stores them
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_stage_full));
            }
#if defined(ATTN_JVP_TRACE) && ATTN_JVP_TRACE >= 2
            if (trace_on && lane == 0 && ((warp - kFirstSoftmaxWarp) & 3) == 0 && it < kTraceSteps) g_trace[20][it] = clock64();    // softmax warp: epilogue ends
#endif
            if (in_range) {
                // L = m + log l (natural log); mu = r / l, plus the constant that was taken out of tS
                const float lse_val = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
                const float mu_val = kHasTQ ? mu + ts_shift : 0.0f;
                const size_t idx = (static_cast<size_t>(b) * args.H + h) * args.Lq + qi;
                if (kSplit) {
                    const size_t pidx = static_cast<size_t>(split) * args.B * args.H * args.Lq + idx;
                    args.part_lse[pidx] = lse_val;
                    args.part_mu[pidx] = mu_val;
                } else {
                    args.lse[idx] = lse_val;
                    if (args.mu != nullptr) args.mu[idx] = mu_val;
                }
            }
            ACC_END(acc_sm_epi);
            g0 += n_kv;
        }
        if (warp == kFirstSoftmaxWarp + ((kMmaWarp - kFirstSoftmaxWarp) & 3)) {   // the softmax warp on the MMA warp's scheduler
            ACC_WRITE(2, acc_sm_scores);
            if (!kEpiWarps) { ACC_WRITE(3, acc_sm_values); ACC_WRITE(4, acc_sm_epi); }
        }
        if (kEpiWarps && warp == kFirstSoftmaxWarp + 4 + ((kMmaWarp - kFirstSoftmaxWarp) & 3)) {   // ... and its epilogue warp
            ACC_WRITE(3, acc_sm_values);
            ACC_WRITE(4, acc_sm_epi);
        }
    }

    // Teardown: every role falls through to here (all waits are bounded).
    // (CTA pair: neither CTA may leave, or free its tensor memory, while the other can still reach into it -- the
    // first CTA's MMAs read and write both, the second CTA's warps arrive on the first one's barriers.)
    tc_fence_before();
    if (kPair) cluster_sync_all(); else __syncthreads();
#ifdef ATTN_JVP_TRACE
    if (trace_on && threadIdx.x == 0) g_trace[kTraceEvents - 1][1] = clock64();      // CTA ends
#endif
    if (warp == kMmaWarp) {
        tc_fence_after();
        if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one warp waits on a barrier on which nothing ever arrives.  The wait
// must give up after its time limit, record ATTN_JVP_ERR_DEVICE_TIMEOUT and let the kernel end normally
// (no trap, no endless loop), leaving the context usable.
// ---------------------------------------------------------------------------------------------
__global__ void bounded_wait_selftest_kernel(int* host_status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int cta_abort;
    if (threadIdx.x == 0) {
        cta_abort = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    AbortState st{&cta_abort, host_status};
    (void)mbar_wait_warp(smem_u32(&bar), 0, st);
}

// ---------------------------------------------------------------------------------------------
// Split-KV merge.  Chunk c of the keys gave (O_c, tO_c, LSE_c, mu_c), each normalised within the chunk.
// With w_c = exp(LSE_c - LSE), LSE = log sum_c exp(LSE_c):
//     O = sum_c w_c O_c,   mu = sum_c w_c mu_c,   tO = sum_c w_c (tO_c + mu_c O_c) - mu O
// (the aggregated form of Appendix C.1 regrouped by chunk; mu = rowsum(P . tS) = d LSE).
// One thread per (row, 4 columns).
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256)
attn_jvp_splitkv_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_to,
                              const float* __restrict__ part_lse, const float* __restrict__ part_mu,
                              __nv_bfloat16* __restrict__ o, __nv_bfloat16* __restrict__ to,
                              float* __restrict__ lse, float* __restrict__ mu,
                              int B, int H, int Lq, int splits, int has_tangent) {
    constexpr int kVecPerRow = D / 4;
    const long long n_rows = static_cast<long long>(B) * Lq * H;
    const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long r = gid / kVecPerRow;             // row index in [B][Lq][H] order
    const int v = static_cast<int>(gid % kVecPerRow);
    if (r >= n_rows) return;
    const int h = static_cast<int>(r % H);
    const long long bl = r / H;
    const int l = static_cast<int>(bl % Lq);
    const int b = static_cast<int>(bl / Lq);
    const size_t stat = (static_cast<size_t>(b) * H + h) * Lq + l;         // index in [B][H][Lq]
    const size_t stat_stride = static_cast<size_t>(B) * H * Lq;
    const size_t vec_stride = static_cast<size_t>(n_rows) * D;

    float lse_max = -INFINITY;
    for (int c = 0; c < splits; ++c) lse_max = fmaxf(lse_max, part_lse[c * stat_stride + stat]);
    float denom = 0.0f;
    for (int c = 0; c < splits; ++c) denom += __expf(part_lse[c * stat_stride + stat] - lse_max);
    const float inv_denom = 1.0f / denom;

    float4 acc_o = make_float4(0.f, 0.f, 0.f, 0.f), acc_t = make_float4(0.f, 0.f, 0.f, 0.f);
    float mu_tot = 0.0f;
    for (int c = 0; c < splits; ++c) {
        const float w = __expf(part_lse[c * stat_stride + stat] - lse_max) * inv_denom;
        const float4 oc = *reinterpret_cast<const float4*>(part_o + c * vec_stride + static_cast<size_t>(r) * D + v * 4);
        acc_o.x = fmaf(w, oc.x, acc_o.x); acc_o.y = fmaf(w, oc.y, acc_o.y);
        acc_o.z = fmaf(w, oc.z, acc_o.z); acc_o.w = fmaf(w, oc.w, acc_o.w);
        if (has_tangent) {
            const float mc = part_mu[c * stat_stride + stat];
            const float4 tc = *reinterpret_cast<const float4*>(part_to + c * vec_stride + static_cast<size_t>(r) * D + v * 4);
            mu_tot = fmaf(w, mc, mu_tot);
            acc_t.x = fmaf(w, fmaf(mc, oc.x, tc.x), acc_t.x); acc_t.y = fmaf(w, fmaf(mc, oc.y, tc.y), acc_t.y);
            acc_t.z = fmaf(w, fmaf(mc, oc.z, tc.z), acc_t.z); acc_t.w = fmaf(w, fmaf(mc, oc.w, tc.w), acc_t.w);
        }
    }
    const size_t out = static_cast<size_t>(r) * D + v * 4;
    uint2 po;
    po.x = pack_bf16(acc_o.x, acc_o.y);
    po.y = pack_bf16(acc_o.z, acc_o.w);
    *reinterpret_cast<uint2*>(o + out) = po;
    if (has_tangent) {
        uint2 pt;
        pt.x = pack_bf16(fmaf(-mu_tot, acc_o.x, acc_t.x), fmaf(-mu_tot, acc_o.y, acc_t.y));
        pt.y = pack_bf16(fmaf(-mu_tot, acc_o.z, acc_t.z), fmaf(-mu_tot, acc_o.w, acc_t.w));
        *reinterpret_cast<uint2*>(to + out) = pt;
    }
    if (v == 0) {
        lse[stat] = lse_max + __logf(denom);
        if (mu != nullptr) mu[stat] = has_tangent ? mu_tot : 0.0f;
    }
}

}  // namespace attn_jvp
