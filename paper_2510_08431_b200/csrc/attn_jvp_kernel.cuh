// Attention-JVP forward kernel for sm_100a (Algorithm 2: FlashAttention-2 forward with JVP).
//
// One CTA owns a 128-row query tile of one (batch, head) and streams the keys in
// tiles of 64.  Roles (warp-specialised, 192 threads):
//   warps 0-3  softmax: one thread per query row; reads S and tS from tensor memory,
//              keeps m, l, r (Algorithm 2 lines 10-12, 16) in registers, writes
//              P~ and H~ = P~ . tS back to tensor memory as bf16 MMA operands,
//              rescales the accumulators when the running max moves, and runs
//              the epilogue (lines 19-23).
//   warp 4     TMA producer: Q,tQ once, then K|tK and V|tV tiles into a shared-memory ring.
//   warp 5     MMA issuer (one thread): tcgen05.mma with accumulators in tensor memory.
//
// Tensor-memory map (512 columns x 128 lanes, fp32):
//   [0, D)        O  accumulator (line 13)
//   [D, 2D)       T = A + B accumulator (lines 14 and 18 share one accumulator, since only
//                 A + B is ever used, line 22)
//   [256+128b, +64)  S  of score buffer b (b = key-tile parity); P~ (bf16) overwrites it
//   [320+128b, +64)  tS of score buffer b;                        H~ (bf16) overwrites it
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
constexpr int kBlockN = 64;         // keys per tile (B_c)
constexpr int kThreads = 192;
constexpr int kSoftmaxThreads = 128;
constexpr int kTmemCols = 512;
constexpr int kScoreCol0 = 256;     // first column of score buffer 0
constexpr int kScoreBufStride = 128;
constexpr float kRescaleThreshold = 8.0f;   // log2 units: rescale only when the max grows by > 2^8
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // bound on every device-side wait

enum Mode : int { kModeJvp = 0, kModeKvTangentFree = 1, kModeFwdOnly = 2 };

// Set by any kernel whose bounded wait expired; later CTAs see it and leave at once.
__device__ int g_abort_flag = 0;

struct KernelArgs {
    __nv_bfloat16* o;
    __nv_bfloat16* to;
    float* lse;
    int* host_status;   // mapped pinned host word, receives the timeout code
    int H, Lq, Lk;
    int n_kv_tiles;
    float scale;        // s
    float scale_log2;   // s * log2(e)
};

template <int D>
struct SmemPlan {
    static constexpr int kHalves = D / 64;                 // 64-element (128-byte) swizzle atoms per row
    static constexpr int kQHalfBytes = kBlockM * 128;      // 16 KB: 128 rows x 128 B
    static constexpr int kQBytes = kHalves * kQHalfBytes;
    static constexpr int kKvHalfBytes = kBlockN * 128;     // 8 KB: 64 rows x 128 B
    static constexpr int kSlotBytes = 2 * kHalves * kKvHalfBytes;  // primal + tangent tile
    static constexpr int kSlots = (D == 128) ? 5 : 8;
    static constexpr int kBytes = 2 * kQBytes + kSlots * kSlotBytes;
    static constexpr int kDynBytes = kBytes + 1024;        // slack for manual 1024-byte alignment
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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

__device__ __noinline__ void report_timeout(const AbortState& st) {
    *st.cta_flag = 1;
    atomicExch(&g_abort_flag, 1);
    if (st.host_status) {
        *reinterpret_cast<volatile int*>(st.host_status) = 10;  // ATTN_JVP_ERR_DEVICE_TIMEOUT
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
                report_timeout(st);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major) {
    return (1u << 4)                       // accumulator format: fp32
         | (1u << 7)                       // A format: bf16
         | (1u << 10)                      // B format: bf16
         | (0u << 15)                      // A: K-major
         | ((b_mn_major ? 1u : 0u) << 16)  // B: K-major or MN-major
         | (static_cast<uint32_t>(n >> 3) << 17)
         | (static_cast<uint32_t>(kBlockM >> 4) << 24);
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (rows x 64 bf16 per swizzle atom): lbo unused.
//   MN-major operand (64 contiguous bf16 along N per atom): lbo = bytes between N atoms.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4)
         | (static_cast<uint64_t>(lbo_bytes >> 4) << 16)
         | (static_cast<uint64_t>(1024u >> 4) << 32)
         | (1ull << 46)     // descriptor version for sm_100
         | (2ull << 61);    // SWIZZLE_128B
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

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int D, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
attn_jvp_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_tq,
                    const __grid_constant__ CUtensorMap tm_tk, const __grid_constant__ CUtensorMap tm_tv,
                    const KernelArgs args) {
    using Plan = SmemPlan<D>;
    constexpr int kHalves = Plan::kHalves;
    constexpr int kSlots = Plan::kSlots;
    constexpr bool kHasTQ = (MODE != kModeFwdOnly);          // tS and T exist
    constexpr bool kHasTKV = (MODE == kModeJvp);             // tK, tV are read

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q_full;
    __shared__ __align__(8) uint64_t bar_slot_full[kSlots];
    __shared__ __align__(8) uint64_t bar_slot_empty[kSlots];
    __shared__ __align__(8) uint64_t bar_s_full[2];
    __shared__ __align__(8) uint64_t bar_p_full[2];
    __shared__ __align__(8) uint64_t bar_pv_done;
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_smem;
    __shared__ int cta_abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int q_tile = blockIdx.x;
    const int h = blockIdx.y;
    const int b = blockIdx.z;
    const int q0 = q_tile * kBlockM;
    const int n_kv = args.n_kv_tiles;

    // An earlier CTA of this (or a previous) launch gave up: do not start.  One thread reads
    // the flag so that the whole CTA takes the same decision.
    if (threadIdx.x == 0) cta_abort = *reinterpret_cast<volatile int*>(&g_abort_flag);
    __syncthreads();
    if (cta_abort != 0) return;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smem_q = smem_base;
    const uint32_t smem_tq = smem_base + Plan::kQBytes;
    const uint32_t smem_ring = smem_base + 2 * Plan::kQBytes;

    AbortState abort_state{&cta_abort, args.host_status};

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar_q_full), 1);
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(smem_u32(&bar_slot_full[i]), 1);
            mbar_init(smem_u32(&bar_slot_empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bar_s_full[i]), 1);
            mbar_init(smem_u32(&bar_p_full[i]), kSoftmaxThreads);
        }
        mbar_init(smem_u32(&bar_pv_done), 1);
        mbar_init(smem_u32(&bar_drain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_smem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == 4 && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        if (kHasTQ) prefetch_tensormap(&tm_tq);
        if (kHasTKV) { prefetch_tensormap(&tm_tk); prefetch_tensormap(&tm_tv); }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_base_smem);
    const uint32_t tmem_o = tmem;
    const uint32_t tmem_t = tmem + D;

    if (warp == 4) {
        // =====================================================================================
        // TMA producer.  Ring order = consumption order: K0, K1, V0, K2, V1, ..., K(n-1), V(n-2), V(n-1).
        // =====================================================================================
        if (lane == 0) {
            constexpr uint32_t kQTx = (kHasTQ ? 2u : 1u) * Plan::kQBytes;
            constexpr uint32_t kKTx = (kHasTKV ? 2u : 1u) * kHalves * Plan::kKvHalfBytes;
            constexpr uint32_t kVTx = kKTx;
            const uint32_t qbar = smem_u32(&bar_q_full);
            mbar_arrive_expect_tx(qbar, kQTx);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
                tma_load_4d(smem_q + hf * Plan::kQHalfBytes, &tm_q, qbar, hf * 64, h, q0, b);
                if (kHasTQ) tma_load_4d(smem_tq + hf * Plan::kQHalfBytes, &tm_tq, qbar, hf * 64, h, q0, b);
            }
            int t = 0;          // ring position
            bool ok = true;
            auto acquire = [&](uint32_t& slot_addr, uint32_t& bar) -> bool {
                const int slot = t % kSlots;
                if (t >= kSlots) {
                    if (!mbar_wait(smem_u32(&bar_slot_empty[slot]), ((t / kSlots) - 1) & 1, abort_state)) return false;
                }
                slot_addr = smem_ring + slot * Plan::kSlotBytes;
                bar = smem_u32(&bar_slot_full[slot]);
                ++t;
                return true;
            };
            auto load_k = [&](int j) -> bool {
                uint32_t dst, bar;
                if (!acquire(dst, bar)) return false;
                mbar_arrive_expect_tx(bar, kKTx);
                // per 64-column half: [K_half (8 KB)][tK_half (8 KB)] so that [K ; tK] is one N = 128 operand
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_4d(dst + hf * 2 * Plan::kKvHalfBytes, &tm_k, bar, hf * 64, h, j * kBlockN, b);
                    if (kHasTKV)
                        tma_load_4d(dst + hf * 2 * Plan::kKvHalfBytes + Plan::kKvHalfBytes, &tm_tk, bar, hf * 64, h, j * kBlockN, b);
                }
                return true;
            };
            auto load_v = [&](int j) -> bool {
                uint32_t dst, bar;
                if (!acquire(dst, bar)) return false;
                mbar_arrive_expect_tx(bar, kVTx);
                // [V_half0][V_half1][tV_half0][tV_half1]: consecutive 64-wide N atoms of [V | tV]
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_4d(dst + hf * Plan::kKvHalfBytes, &tm_v, bar, hf * 64, h, j * kBlockN, b);
                    if (kHasTKV)
                        tma_load_4d(dst + (kHalves + hf) * Plan::kKvHalfBytes, &tm_tv, bar, hf * 64, h, j * kBlockN, b);
                }
                return true;
            };
            ok = load_k(0);
            for (int j = 0; ok && j < n_kv; ++j) {
                if (j + 1 < n_kv) ok = load_k(j + 1);
                if (ok) ok = load_v(j);
            }
            if (!ok) {
                // Abandoning the tile: let the copies already in flight land before the CTA exits.
                const int issued = t;
                for (int u = (issued > kSlots ? issued - kSlots : 0); u < issued; ++u) {
                    const uint32_t bar = smem_u32(&bar_slot_full[u % kSlots]);
                    const uint32_t par = (u / kSlots) & 1;
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar, par) && globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 5) {
        // =====================================================================================
        // MMA issuer (a single thread issues every tcgen05.mma and the commits that track them).
        // =====================================================================================
        if (lane == 0) {
            constexpr uint32_t kIdescS1 = make_idesc(kHasTKV ? 2 * kBlockN : kBlockN, false);  // Q x [K;tK] or Q x K
            constexpr uint32_t kIdescS2 = make_idesc(kBlockN, false);                          // tQ x K
            constexpr uint32_t kIdescPV = make_idesc(kHasTKV ? 2 * D : D, true);               // P~ x [V|tV] or P~ x V
            constexpr uint32_t kIdescHV = make_idesc(D, true);                                 // H~ x V
            constexpr uint32_t kVLbo = Plan::kKvHalfBytes;   // bytes between 64-wide N atoms of a V slot
            int t = 0;
            bool ok = mbar_wait(smem_u32(&bar_q_full), 0, abort_state);

            auto wait_slot = [&](uint32_t& slot_addr, uint32_t& empty_bar) -> bool {
                const int slot = t % kSlots;
                if (!mbar_wait(smem_u32(&bar_slot_full[slot]), (t / kSlots) & 1, abort_state)) return false;
                slot_addr = smem_ring + slot * Plan::kSlotBytes;
                empty_bar = smem_u32(&bar_slot_empty[slot]);
                ++t;
                return true;
            };
            auto issue_scores = [&](int j) -> bool {
                uint32_t ks, empty_bar;
                if (!wait_slot(ks, empty_bar)) return false;
                tc_fence_after();
                const uint32_t tm_s = tmem + kScoreCol0 + (j & 1) * kScoreBufStride;
                const uint32_t tm_ts = tm_s + kBlockN;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t koff = (k / 4) * Plan::kQHalfBytes + (k % 4) * 32;
                    const uint32_t boff = (k / 4) * 2 * Plan::kKvHalfBytes + (k % 4) * 32;
                    mma_ss(tm_s, make_smem_desc(smem_q + koff, 16), make_smem_desc(ks + boff, 16), kIdescS1, k > 0);
                }
                if (kHasTQ) {
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t koff = (k / 4) * Plan::kQHalfBytes + (k % 4) * 32;
                        const uint32_t boff = (k / 4) * 2 * Plan::kKvHalfBytes + (k % 4) * 32;
                        mma_ss(tm_ts, make_smem_desc(smem_tq + koff, 16), make_smem_desc(ks + boff, 16), kIdescS2,
                               (kHasTKV || k > 0) ? 1u : 0u);
                    }
                }
                tc_commit(empty_bar);
                tc_commit(smem_u32(&bar_s_full[j & 1]));
                return true;
            };
            auto issue_values = [&](int j) -> bool {
                uint32_t vs, empty_bar;
                if (!wait_slot(vs, empty_bar)) return false;
                if (!mbar_wait(smem_u32(&bar_p_full[j & 1]), (j >> 1) & 1, abort_state)) return false;
                tc_fence_after();
                const uint32_t tm_p = tmem + kScoreCol0 + (j & 1) * kScoreBufStride;
                const uint32_t tm_h = tm_p + kBlockN;
#pragma unroll
                for (int k = 0; k < kBlockN / 16; ++k) {
                    mma_ts(tmem_o, tm_p + k * 8, make_smem_desc(vs + k * 2048, kVLbo), kIdescPV, (j > 0 || k > 0) ? 1u : 0u);
                }
                if (kHasTQ) {
#pragma unroll
                    for (int k = 0; k < kBlockN / 16; ++k) {
                        mma_ts(tmem_t, tm_h + k * 8, make_smem_desc(vs + k * 2048, kVLbo), kIdescHV,
                               (kHasTKV || j > 0 || k > 0) ? 1u : 0u);
                    }
                }
                tc_commit(empty_bar);
                tc_commit(smem_u32(&bar_pv_done));
                return true;
            };

            if (ok) ok = issue_scores(0);
            for (int j = 0; ok && j < n_kv; ++j) {
                if (j + 1 < n_kv) ok = issue_scores(j + 1);
                if (ok) ok = issue_values(j);
            }
            if (!ok) {
                // Abandoning the tile: wait (bounded) until the tensor core has drained what was issued.
                tc_commit(smem_u32(&bar_drain));
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(smem_u32(&bar_drain), 0) && globaltimer_ns() - t0 < 100000000ull) {}
            }
        }
    } else {
        // =====================================================================================
        // Softmax warps: thread r owns query row q0 + r (tensor-memory lane r).
        // =====================================================================================
        const int row = threadIdx.x;                       // 0..127
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        const float c1 = args.scale_log2;
        const float sc = args.scale;
        const bool neg_scale = c1 < 0.0f;
        float m_ref = -INFINITY;   // running reference max, log2 domain (m of Algorithm 2, lazily updated)
        float l_run = 0.0f;        // l
        float r_run = 0.0f;        // r (of the centred tS, see below)
        float ts_shift = 0.0f;     // per-row constant subtracted from tS
        bool ok = true;

        for (int j = 0; j < n_kv; ++j) {
            const int bsel = j & 1;
            if (!mbar_wait(smem_u32(&bar_s_full[bsel]), (j >> 1) & 1, abort_state)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tm_s = tmem + lane_base + kScoreCol0 + bsel * kScoreBufStride;
            const uint32_t tm_ts = tm_s + kBlockN;

            uint32_t sv[64];
            uint32_t tv[64];
            TMEM_LD32(tm_s, sv, 0);
            TMEM_LD32(tm_s + 32, sv, 32);
            if (kHasTQ) {
                TMEM_LD32(tm_ts, tv, 0);
                TMEM_LD32(tm_ts + 32, tv, 32);
            }
            tc_wait_ld();

            // keys past Lk (zero-filled by TMA) must not enter the softmax
            const int valid = args.Lk - j * kBlockN;
            if (valid < kBlockN) {
                const uint32_t masked = neg_scale ? 0x7F800000u : 0xFF800000u;   // -inf after scaling
#pragma unroll
                for (int c = 0; c < 64; ++c) if (c >= valid) sv[c] = masked;
            }

            // rowmax(S_ij) in the log2 domain
            float mx = __uint_as_float(sv[0]);
            if (!neg_scale) {
#pragma unroll
                for (int c = 1; c < 64; ++c) mx = fmaxf(mx, __uint_as_float(sv[c]));
            } else {
#pragma unroll
                for (int c = 1; c < 64; ++c) mx = fminf(mx, __uint_as_float(sv[c]));
            }
            mx *= c1;

            // m_new = max(m, rowmax), applied lazily: the result does not depend on which
            // reference is used as long as exp() stays in range.
            float alpha = 1.0f;
            const bool need = mx > m_ref + kRescaleThreshold;
            if (need) {
                alpha = ex2f(m_ref - mx);    // e^{m - m_new}; 0 on the first tile (m = -inf)
                m_ref = mx;
            }
            if (j > 0 && __any_sync(0xffffffffu, need)) {
                // the accumulators must be complete up to tile j-1 before they are rescaled
                if (!mbar_wait(smem_u32(&bar_pv_done), (j - 1) & 1, abort_state)) { ok = false; break; }
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
            }
            l_run *= alpha;
            r_run *= alpha;

            // P~ = exp(S - m_new), l += rowsum(P~)
            float lsum = 0.0f;
#pragma unroll
            for (int c = 0; c < 64; ++c) {
                const float p = ex2f(fmaf(__uint_as_float(sv[c]), c1, -m_ref));
                sv[c] = __float_as_uint(p);
                lsum += p;
            }
            if (valid < kBlockN) {
                // exact zeros for masked keys whatever the scale (0 * inf above would give NaN)
                lsum = 0.0f;
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    if (c >= valid) sv[c] = 0u;
                    lsum += __uint_as_float(sv[c]);
                }
            }
            l_run += lsum;
            {
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) pk[c] = pack_bf16(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1]));
                TMEM_ST32(tm_s, pk, 0);
            }
            if (kHasTQ) {
                // tO does not change when a per-row constant is subtracted from tS (softmax is shift
                // invariant: the constant leaves H~ V - (r/l) O unchanged).  Centring tS on its P-weighted
                // mean over the first tile keeps H~ and r small, so that the bf16 rounding of H~ scales
                // with |tS - mu| instead of |tS| when the two terms cancel in the epilogue.
                if (j == 0) {
                    float num = 0.0f;
#pragma unroll
                    for (int c = 0; c < 64; ++c) num = fmaf(__uint_as_float(sv[c]), __uint_as_float(tv[c]) * sc, num);
                    ts_shift = num / lsum;
                }
                // H~ = P~ . tS, r += rowsum(H~)
                float rsum = 0.0f;
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    const float hv = __uint_as_float(sv[c]) * fmaf(__uint_as_float(tv[c]), sc, -ts_shift);
                    tv[c] = __float_as_uint(hv);
                    rsum += hv;
                }
                r_run += rsum;
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) pk[c] = pack_bf16(__uint_as_float(tv[2 * c]), __uint_as_float(tv[2 * c + 1]));
                TMEM_ST32(tm_ts, pk, 0);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bar_p_full[bsel]));
        }

        // Epilogue: O/l, L = m + log l, tO = (T - r (O/l)) / l
        // A parity wait can only tell the current phase from the previous one, and the value MMAs of
        // tile n-2 may still be running here: wait for them first, then for those of tile n-1.
        if (ok && n_kv >= 2) ok = mbar_wait(smem_u32(&bar_pv_done), (n_kv - 2) & 1, abort_state);
        if (ok) ok = mbar_wait(smem_u32(&bar_pv_done), (n_kv - 1) & 1, abort_state);
        if (ok) {
            tc_fence_after();
            const int qi = q0 + row;
            const bool in_range = qi < args.Lq;
            const float inv_l = 1.0f / l_run;
            const float mu = r_run * inv_l;
            const size_t row_off = ((static_cast<size_t>(b) * args.Lq + (in_range ? qi : 0)) * args.H + h) * D;
            __nv_bfloat16* o_row = args.o + row_off;
            __nv_bfloat16* to_row = kHasTQ ? args.to + row_off : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t ov[32];
                uint32_t tvv[32];
                TMEM_LD32(tmem_o + lane_base + c0, ov, 0);
                if (kHasTQ) TMEM_LD32(tmem_t + lane_base + c0, tvv, 0);
                tc_wait_ld();
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
                if (in_range) {
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        *reinterpret_cast<uint4*>(o_row + c0 + v4 * 8) = make_uint4(po[4 * v4], po[4 * v4 + 1], po[4 * v4 + 2], po[4 * v4 + 3]);
                        if (kHasTQ)
                            *reinterpret_cast<uint4*>(to_row + c0 + v4 * 8) = make_uint4(pt[4 * v4], pt[4 * v4 + 1], pt[4 * v4 + 2], pt[4 * v4 + 3]);
                    }
                }
            }
            if (in_range) {
                args.lse[(static_cast<size_t>(b) * args.H + h) * args.Lq + qi] = (m_ref + log2f(l_run)) * 0.6931471805599453f;
            }
        }
    }

    // Teardown: every role falls through to here (all waits are bounded).
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace attn_jvp
