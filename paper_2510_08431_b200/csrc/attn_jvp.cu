// Host side of the attention-JVP library: argument validation, TMA tensor maps, launch.
// The C ABI is declared in include/attn_jvp.h.
#include "attn_jvp.h"

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>

#include "attn_jvp_kernel.cuh"
#include "qknorm_jvp.cuh"

namespace {

using attn_jvp::KernelArgs;

constexpr int kVersion = 100;   // 0.1.0
constexpr int kMaxDevices = 64;
constexpr int kPersistentMaxTiles = 128;   // key tiles per work item up to which CTAs are persistent

thread_local cudaStream_t tl_stream = nullptr;
thread_local char tl_cuda_msg[256] = "";
thread_local char tl_strerror_buf[384];

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Lazily initialised per-device state.  Several host threads may make their first call at the same time (the
// stream of attn_jvp_fwd is per thread): every slow path below runs under `lock`, and what the fast paths read is
// published through atomics only when complete.
struct DeviceState {
    std::mutex lock;
    std::atomic<int> cc_major{0};                 // 0 = not queried yet
    int sm_count = 0;                             // valid once cc_major != 0
    int smem_optin = 0;                           // valid once cc_major != 0
    std::atomic<int*> host_status{nullptr};       // mapped pinned host word ...
    std::atomic<int*> host_status_dev{nullptr};   // ... and its device-side address (published first)
    std::atomic<bool> unwatched_launch{false};    // a kernel ran here before the status word existed
    std::atomic<int> dyn_smem[2][3][2][2];        // dynamic shared memory per kernel instantiation, 0 = not set up
    std::atomic<int> dyn_smem_pair[3][2];         // ... of the CTA-pair kernels
    std::atomic<void*> static_scratch{nullptr};   // device address of the built-in scratch array
};
DeviceState g_dev[kMaxDevices];
std::mutex g_encode_lock;
std::atomic<EncodeTiledFn> g_encode_tiled{nullptr};

// Tuning knobs (attn_jvp_set_tuning); 0 = the library's own choice.
std::atomic<int> g_tune_softmax_groups{0};
std::atomic<int> g_tune_cta_pair{0};

// Softmax groups of the CTA-pair kernel (measured: with tangents one group is 3-8 % faster than two there as well;
// the forward-only pair is 14 % faster with two).
int softmax_groups_for_pair(int mode) {
    const int forced = g_tune_softmax_groups.load(std::memory_order_relaxed);
    if (forced == 1 || forced == 2) return forced;
    return mode == attn_jvp::kModeFwdOnly ? 2 : 1;
}

// Whether a call runs on the CTA-pair kernel (clusters of two CTAs sharing the K/V operand tiles and one MMA
// instruction stream).  It exists at D = 128, without key chunks.
bool use_cta_pair(int mode, int D, bool split, int tiles_per_item) {
    if (D != 128 || split) return false;
    const int forced = g_tune_cta_pair.load(std::memory_order_relaxed);
    if (forced == 1) return false;
    if (forced == 2) return true;
    // Measured on B200.  Full JVP: 2-20 % faster than one CTA per query tile from about eight key tiles per item on
    // (12 % on the 32760-token self-attention workloads), slower with fewer.  Tangent-free K/V: 4-20 % faster from
    // two key tiles per item on (6 % on the 512-key cross-attention workload, 9 % at 32760 keys).  Forward only:
    // 4-9 % slower than one CTA per query tile with two softmax groups at every length tried (64 to 32760 keys).
    if (mode == attn_jvp::kModeJvp) return tiles_per_item >= 6;
    if (mode == attn_jvp::kModeKvTangentFree) return tiles_per_item >= 2;
    return false;
}

// Softmax warpgroups per CTA for a kernel variant: two groups take alternate key tiles, which pays where the
// softmax arithmetic, not the tensor pipe, sets the pace of a key tile.
int softmax_groups_for(int mode, int D, int tiles_per_item) {
    const int forced = g_tune_softmax_groups.load(std::memory_order_relaxed);
    if (forced == 1 || forced == 2) return forced;
    // Measured on B200 (image- and video-length self-attention): at D = 64 the tensor work per key tile is half
    // that of D = 128 while the softmax work is the same, and two groups are 1.1-1.3x faster in every mode.  At
    // D = 128 the forward-only mode (a third of the tensor work of the JVP per tile) is 2-14 % faster with two
    // groups from eight key tiles per item on; with tangents one group is as fast or faster.
    if (D == 64) return 2;
    return (mode == attn_jvp::kModeFwdOnly && tiles_per_item >= 8) ? 2 : 1;
}

int cuda_fail(const char* what, cudaError_t e) {
    snprintf(tl_cuda_msg, sizeof tl_cuda_msg, "%s: %s", what, cudaGetErrorString(e));
    return ATTN_JVP_ERR_CUDA;
}

int get_encode_fn() {
    if (g_encode_tiled.load(std::memory_order_acquire)) return 0;
    std::lock_guard<std::mutex> guard(g_encode_lock);
    if (g_encode_tiled.load(std::memory_order_relaxed)) return 0;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return cuda_fail("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", e);
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        snprintf(tl_cuda_msg, sizeof tl_cuda_msg, "cuTensorMapEncodeTiled not available from this driver");
        return ATTN_JVP_ERR_CUDA;
    }
    g_encode_tiled.store(reinterpret_cast<EncodeTiledFn>(fn), std::memory_order_release);
    return 0;
}

// The current device, checked to be sm_100; its attributes are queried once.  Enqueues nothing.
int current_device(int* dev_out, DeviceState** st_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail("cudaGetDevice", e);
    if (dev < 0 || dev >= kMaxDevices) return ATTN_JVP_ERR_ARCH;
    DeviceState& st = g_dev[dev];
    if (st.cc_major.load(std::memory_order_acquire) == 0) {
        std::lock_guard<std::mutex> guard(st.lock);
        if (st.cc_major.load(std::memory_order_relaxed) == 0) {
            int major = 0, sms = 0, optin = 0;
            e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
            if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute(ComputeCapabilityMajor)", e);
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute(MultiProcessorCount)", e);
            e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
            if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute(MaxSharedMemoryPerBlockOptin)", e);
            st.sm_count = sms;
            st.smem_optin = optin;
            st.cc_major.store(major > 0 ? major : -1, std::memory_order_release);
        }
    }
    if (st.cc_major.load(std::memory_order_acquire) != 10) return ATTN_JVP_ERR_ARCH;
    *dev_out = dev;
    *st_out = &st;
    return 0;
}

// The pinned status word a kernel writes its timeout code to; allocated on the first call that may allocate.
int ensure_status_word(DeviceState& st) {
    if (st.host_status.load(std::memory_order_acquire)) return 0;
    std::lock_guard<std::mutex> guard(st.lock);
    if (st.host_status.load(std::memory_order_relaxed)) return 0;
    int* hp = nullptr;
    cudaError_t e = cudaHostAlloc((void**)&hp, sizeof(int), cudaHostAllocMapped);
    if (e != cudaSuccess) return cuda_fail("cudaHostAlloc(status word)", e);
    *hp = 0;
    int* dp = nullptr;
    e = cudaHostGetDevicePointer((void**)&dp, hp, 0);
    if (e != cudaSuccess) { cudaFreeHost(hp); return cuda_fail("cudaHostGetDevicePointer", e); }
    st.host_status_dev.store(dp, std::memory_order_release);   // a reader that sees the host pointer sees this one too
    st.host_status.store(hp, std::memory_order_release);
    return 0;
}

// bf16 [B][L][H][D] tensor seen as a rank-4 map {D, H, L, B}; one box = 64 columns x `rows` rows
// of one head, laid out in shared memory with the 128-byte swizzle the MMA descriptors expect.
int make_map(CUtensorMap* map, const void* base, int B, int L, int H, int D, int rows) {
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2, (cuuint64_t)L * H * D * 2};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)rows, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = g_encode_tiled.load(std::memory_order_acquire)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(tl_cuda_msg, sizeof tl_cuda_msg, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return ATTN_JVP_ERR_CUDA;
    }
    return 0;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + nb && b0 < a0 + na;
}

template <int D, int MODE, bool SPLIT, int GROUPS, bool PAIR = false>
int launch(const CUtensorMap* maps, const KernelArgs& ka, dim3 grid, cudaStream_t stream, DeviceState& st) {
    auto kern = attn_jvp::attn_jvp_fwd_kernel<D, MODE, SPLIT, GROUPS, PAIR>;
    using Plan = attn_jvp::SmemPlan<D, MODE, GROUPS, PAIR, SPLIT>;
    std::atomic<int>& slot = PAIR ? st.dyn_smem_pair[MODE][GROUPS - 1] : st.dyn_smem[D == 128][MODE][SPLIT][GROUPS - 1];
    int smem = slot.load(std::memory_order_acquire);
    if (smem == 0) {
        // dynamic shared memory = the operand layout (declared 1024-byte aligned in the kernel) plus the exchange
        // area of two softmax groups; it must fit beside the kernel's static shared memory
        std::lock_guard<std::mutex> guard(st.lock);
        smem = slot.load(std::memory_order_relaxed);
        if (smem == 0) {
            cudaFuncAttributes fa;
            cudaError_t e = cudaFuncGetAttributes(&fa, kern);
            if (e != cudaSuccess) return cuda_fail("cudaFuncGetAttributes", e);
            const int want = Plan::kDynBytes;
            const int room = st.smem_optin - (int)fa.sharedSizeBytes;
            if (want > room) {
                snprintf(tl_cuda_msg, sizeof tl_cuda_msg, "device offers %d bytes of shared memory, kernel needs %d",
                         room, want);
                return ATTN_JVP_ERR_CUDA;
            }
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, want);
            if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute(MaxDynamicSharedMemorySize)", e);
            smem = want;
            slot.store(want, std::memory_order_release);
        }
    }
    if (PAIR) {
        // clusters of two CTAs (the two SMs of a TPC); the grid holds an even number of CTAs
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(attn_jvp::num_threads(GROUPS), 1, 1);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, kern, maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], maps[6],
                                           maps[7], maps[8], ka);
        if (e != cudaSuccess) return cuda_fail("cluster kernel launch", e);
        return 0;
    }
    kern<<<grid, attn_jvp::num_threads(GROUPS), smem, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], maps[6],
                                                     maps[7], maps[8], ka);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail("kernel launch", e);
    return 0;
}

// Bytes of scratch the split-KV path needs: per chunk fp32 O and tO partials ([B][Lq][H][D]) and fp32 LSE and mu
// partials ([B][H][Lq], each padded to a multiple of 16 bytes).
struct SplitLayout {
    size_t vec_bytes;    // one chunk set of O (or tO) partials, all chunks
    size_t stat_bytes;   // one chunk set of LSE (or mu) partials, all chunks, padded
    size_t total;
};
SplitLayout split_layout(int B, int H, int Lq, int D, int splits) {
    SplitLayout L;
    L.vec_bytes = (size_t)splits * B * Lq * H * D * sizeof(float);
    L.stat_bytes = (((size_t)splits * B * H * Lq * sizeof(float)) + 15) & ~(size_t)15;
    L.total = 2 * L.vec_bytes + 2 * L.stat_bytes;
    return L;
}
// Chunks actually used for `splits` requested chunks: whole 64-key tiles per chunk, no empty chunk.
void split_plan(int Lk, int splits, int* tiles_per_split, int* eff_splits) {
    const int n_tiles = (Lk + attn_jvp::kBlockN - 1) / attn_jvp::kBlockN;
    if (splits > n_tiles) splits = n_tiles;
    const int tps = (n_tiles + splits - 1) / splits;
    *tiles_per_split = tps;
    *eff_splits = (n_tiles + tps - 1) / tps;
}

int run(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
        void* o, void* to, float* lse, float* mu, int B, int H, int Lq, int Lk, int D, float scale, unsigned flags,
        int splits, void* workspace, size_t workspace_bytes, cudaStream_t stream, bool may_allocate = true) {
    // ---- validation: nothing is enqueued unless everything checks out ----
    if (flags & ~(ATTN_JVP_KV_TANGENT_FREE | ATTN_JVP_FWD_ONLY)) return ATTN_JVP_ERR_FLAGS;
    const bool fwd_only = (flags & ATTN_JVP_FWD_ONLY) != 0;
    const bool kv_free = (flags & ATTN_JVP_KV_TANGENT_FREE) != 0;
    const int mode = fwd_only ? attn_jvp::kModeFwdOnly : (kv_free ? attn_jvp::kModeKvTangentFree : attn_jvp::kModeJvp);
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1) return ATTN_JVP_ERR_SHAPE;
    if (D != 64 && D != 128) return ATTN_JVP_ERR_UNSUPPORTED_D;
    const long double nq = (long double)B * H * Lq * D, nk = (long double)B * H * Lk * D;
    if (nq * 2 > 9.0e18L || nk * 2 > 9.0e18L) return ATTN_JVP_ERR_SHAPE;
    if (!q || !k || !v || !o || !lse) return ATTN_JVP_ERR_NULL;
    if (!fwd_only && (!tq || !to)) return ATTN_JVP_ERR_NULL;
    if (mode == attn_jvp::kModeJvp && (!tk || !tv)) return ATTN_JVP_ERR_NULL;
    if (!std::isfinite(scale)) return ATTN_JVP_ERR_SCALE;
    if (splits < 1 || splits > 1024) return ATTN_JVP_ERR_SHAPE;
    int tiles_per_split = 0, eff_splits = 1;
    split_plan(Lk, splits, &tiles_per_split, &eff_splits);
    const bool split = eff_splits > 1;
    // work items = query tiles x heads x batch x chunks; item + gridDim.x must not overflow an int in the kernel
    const long long n_q_tiles = (Lq + attn_jvp::kBlockM - 1) / attn_jvp::kBlockM;
    const long double n_items_ld = (long double)n_q_tiles * H * B * eff_splits;
    if (n_items_ld > (long double)(0x7fffffffLL - 65536)) return ATTN_JVP_ERR_SHAPE;
    const long long n_items = n_q_tiles * H * B * eff_splits;
    SplitLayout lay = split_layout(B, H, Lq, D, eff_splits);
    if (split) {
        if (!workspace) return ATTN_JVP_ERR_NULL;
        if ((uintptr_t)workspace & 15u) return ATTN_JVP_ERR_ALIGN;
        if (workspace_bytes < lay.total) return ATTN_JVP_ERR_WORKSPACE;
    }
    const void* used_in[6] = {q, k, v, fwd_only ? nullptr : tq, mode == attn_jvp::kModeJvp ? tk : nullptr,
                              mode == attn_jvp::kModeJvp ? tv : nullptr};
    void* used_out[5] = {o, fwd_only ? nullptr : to, lse, mu, split ? workspace : nullptr};
    for (const void* p : used_in) if (p && ((uintptr_t)p & 15u)) return ATTN_JVP_ERR_ALIGN;
    for (const void* p : used_out) if (p && ((uintptr_t)p & 15u)) return ATTN_JVP_ERR_ALIGN;
    const size_t q_bytes = (size_t)B * Lq * H * D * 2, k_bytes = (size_t)B * Lk * H * D * 2;
    const size_t lse_bytes = (size_t)B * H * Lq * 4;
    const size_t in_bytes[6] = {q_bytes, k_bytes, k_bytes, q_bytes, k_bytes, k_bytes};
    const size_t out_bytes[5] = {q_bytes, q_bytes, lse_bytes, lse_bytes, lay.total};
    for (int a = 0; a < 5; ++a) {
        for (int i = 0; i < 6; ++i)
            if (overlaps(used_out[a], out_bytes[a], used_in[i], in_bytes[i])) return ATTN_JVP_ERR_ALIAS;
        for (int c = a + 1; c < 5; ++c)
            if (overlaps(used_out[a], out_bytes[a], used_out[c], out_bytes[c])) return ATTN_JVP_ERR_ALIAS;
    }

    int dev = 0;
    DeviceState* stp = nullptr;
    if (int rc = current_device(&dev, &stp)) return rc;
    DeviceState& st = *stp;
    if (int rc = get_encode_fn()) return rc;
    if (may_allocate) {
        if (int rc = ensure_status_word(st)) return rc;
    }
    cudaError_t e;

    // ---- which kernel variant (decided on the number of 64-key tiles per item), and its key-tile size ----
    const int tiles64 = (Lk + attn_jvp::kBlockN - 1) / attn_jvp::kBlockN;
    const int tiles_per_item = split ? tiles_per_split : tiles64;
    const bool pair = use_cta_pair(mode, D, split, tiles_per_item);
    const int key_tile = attn_jvp::key_tile(D, mode, split, pair);

    // ---- tensor maps (Q-side boxes are 128 rows, K-side boxes one key tile) ----
    CUtensorMap maps[9];
    if (int rc = make_map(&maps[0], q, B, Lq, H, D, attn_jvp::kBlockM)) return rc;
    if (int rc = make_map(&maps[1], k, B, Lk, H, D, key_tile)) return rc;
    if (int rc = make_map(&maps[2], v, B, Lk, H, D, key_tile)) return rc;
    if (int rc = make_map(&maps[3], fwd_only ? q : tq, B, Lq, H, D, attn_jvp::kBlockM)) return rc;
    if (int rc = make_map(&maps[4], mode == attn_jvp::kModeJvp ? tk : k, B, Lk, H, D, key_tile)) return rc;
    if (int rc = make_map(&maps[5], mode == attn_jvp::kModeJvp ? tv : v, B, Lk, H, D, key_tile)) return rc;
    // output tiles (bf16, stored from shared memory by TMA; the split-KV kernel does not use these two)
    if (int rc = make_map(&maps[6], o, B, Lq, H, D, attn_jvp::kBlockM)) return rc;
    if (int rc = make_map(&maps[7], fwd_only ? o : to, B, Lq, H, D, attn_jvp::kBlockM)) return rc;
    // K once more with boxes of half a key tile (the CTA-pair kernel splits the operand of tQ K^T by rows)
    if (int rc = make_map(&maps[8], k, B, Lk, H, D, attn_jvp::kBlockN / 2)) return rc;

    KernelArgs ka;
    ka.o = reinterpret_cast<__nv_bfloat16*>(o);
    ka.to = reinterpret_cast<__nv_bfloat16*>(to);
    ka.lse = lse;
    ka.host_status = st.host_status_dev.load(std::memory_order_acquire);
    // no status word yet (only the allocation-free entry point has run here): the device-side flag is the only record
    if (ka.host_status == nullptr) st.unwatched_launch.store(true, std::memory_order_release);
    ka.H = H;
    ka.Lq = Lq;
    ka.Lk = Lk;
    ka.n_kv_tiles = (Lk + key_tile - 1) / key_tile;
    ka.scale = scale;
    // The kernel masks the keys past Lk by setting their scaled score to -inf, which needs a nonzero factor: a zero
    // scale (every score 0) is computed with 2^-100 in the exponent, which changes no result bit (tS keeps the 0).
    ka.scale_log2 = (scale == 0.0f) ? 0x1p-100f : scale * 1.4426950408889634f;
    ka.mu = mu;
    ka.B = B;
    ka.splits = eff_splits;
    ka.tiles_per_split = tiles_per_split;
    ka.part_o = ka.part_to = ka.part_lse = ka.part_mu = nullptr;
    if (split) {
        char* w = static_cast<char*>(workspace);
        ka.part_o = reinterpret_cast<float*>(w);
        ka.part_to = reinterpret_cast<float*>(w + lay.vec_bytes);
        ka.part_lse = reinterpret_cast<float*>(w + 2 * lay.vec_bytes);
        ka.part_mu = reinterpret_cast<float*>(w + 2 * lay.vec_bytes + lay.stat_bytes);
    }

    // persistent CTAs: one per SM (fewer if there is less work), sharing the work items round-robin
    ka.n_q_tiles = (int)n_q_tiles;
    ka.n_items = (int)n_items;
    // Short items (few key tiles): one persistent CTA per SM, so that the epilogue of an item overlaps the
    // start of the next.  Long items: one CTA per item, which lets the hardware balance the load (a static
    // round-robin costs up to one item of imbalance at the end, which is more than the overlap saves there).
    const bool persistent = tiles_per_item <= kPersistentMaxTiles;
    int rc;
    if (pair) {
        // A work item is a 256-row query block (two tiles, one per CTA of a pair); with an odd number of tiles the
        // last pair's second CTA has no rows and writes nothing.
        const long long n_q_pairs = (n_q_tiles + 1) / 2;
        const long long n_pair_items = n_q_pairs * H * B;
        ka.n_q_tiles = (int)n_q_pairs;
        ka.n_items = (int)n_pair_items;
        const long long max_pairs = st.sm_count / 2;
        const long long n_pairs = (persistent && n_pair_items > max_pairs) ? max_pairs : n_pair_items;
        const dim3 pair_grid((unsigned)(2 * n_pairs), 1, 1);
        const bool two = softmax_groups_for_pair(mode) == 2;
        switch (mode) {
            case attn_jvp::kModeJvp:
                return two ? launch<128, attn_jvp::kModeJvp, false, 2, true>(maps, ka, pair_grid, stream, st)
                           : launch<128, attn_jvp::kModeJvp, false, 1, true>(maps, ka, pair_grid, stream, st);
            case attn_jvp::kModeKvTangentFree:
                return two ? launch<128, attn_jvp::kModeKvTangentFree, false, 2, true>(maps, ka, pair_grid, stream, st)
                           : launch<128, attn_jvp::kModeKvTangentFree, false, 1, true>(maps, ka, pair_grid, stream, st);
            default:
                return two ? launch<128, attn_jvp::kModeFwdOnly, false, 2, true>(maps, ka, pair_grid, stream, st)
                           : launch<128, attn_jvp::kModeFwdOnly, false, 1, true>(maps, ka, pair_grid, stream, st);
        }
    }
    const long long n_ctas = (persistent && n_items > st.sm_count) ? st.sm_count : n_items;
    const dim3 grid((unsigned)n_ctas, 1, 1);
    const int groups = softmax_groups_for(mode, D, tiles_per_item);
#define ATTN_JVP_DISPATCH_G(DD, SS, GG)                                                                            \
    switch (mode) {                                                                                               \
        case attn_jvp::kModeJvp: rc = launch<DD, attn_jvp::kModeJvp, SS, GG>(maps, ka, grid, stream, st); break;   \
        case attn_jvp::kModeKvTangentFree:                                                                        \
            rc = launch<DD, attn_jvp::kModeKvTangentFree, SS, GG>(maps, ka, grid, stream, st); break;              \
        default: rc = launch<DD, attn_jvp::kModeFwdOnly, SS, GG>(maps, ka, grid, stream, st); break;               \
    }
#define ATTN_JVP_DISPATCH(DD, SS)                                                                                  \
    if (groups == 2) { ATTN_JVP_DISPATCH_G(DD, SS, 2) } else { ATTN_JVP_DISPATCH_G(DD, SS, 1) }
    if (D == 128) {
        if (split) { ATTN_JVP_DISPATCH(128, true) } else { ATTN_JVP_DISPATCH(128, false) }
    } else {
        if (split) { ATTN_JVP_DISPATCH(64, true) } else { ATTN_JVP_DISPATCH(64, false) }
    }
#undef ATTN_JVP_DISPATCH_G
#undef ATTN_JVP_DISPATCH
    if (rc != 0 || !split) return rc;

    // merge the chunks (same stream: ordered after the partial kernel)
    const long long n_threads = (long long)B * Lq * H * (D / 4);
    const unsigned blocks = (unsigned)((n_threads + 255) / 256);
    if (D == 128)
        attn_jvp::attn_jvp_splitkv_merge_kernel<128><<<blocks, 256, 0, stream>>>(
            ka.part_o, ka.part_to, ka.part_lse, ka.part_mu, ka.o, ka.to, lse, mu, B, H, Lq, eff_splits, fwd_only ? 0 : 1);
    else
        attn_jvp::attn_jvp_splitkv_merge_kernel<64><<<blocks, 256, 0, stream>>>(
            ka.part_o, ka.part_to, ka.part_lse, ka.part_mu, ka.o, ka.to, lse, mu, B, H, Lq, eff_splits, fwd_only ? 0 : 1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail("merge kernel launch", e);
    return 0;
}


// ---------------------------------------------------------------------------------------------
// Host-buffer pipeline: the heads are processed in groups; while the kernel works on one group, the copy
// engines bring in the next group's inputs and take out the previous group's outputs.
// ---------------------------------------------------------------------------------------------
// Buffer sets of the host pipeline: with three, the copy-in of group g + 2 no longer waits for the copy-out of
// group g (with two sets a stage took copy-in + copy-out, 10.7 ms on the headline shape, instead of the kernel's 9.2).
constexpr int kHostSets = 3;
struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, comp = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, in_done[kHostSets] = {}, comp_done[kHostSets] = {}, out_done[kHostSets] = {},
                end_in = nullptr, end_comp = nullptr, end_out = nullptr;
    std::mutex lock;     // one enqueue at a time per device: the events are reused from call to call
};
HostPipe g_host_pipe[kMaxDevices];

// Creates the pipeline's streams and events; on failure everything created so far is released again.
int host_pipe_setup(HostPipe& hp) {
    if (hp.ready) return 0;
    cudaStream_t* streams[3] = {&hp.in, &hp.comp, &hp.out};
    cudaEvent_t* events[4 + 3 * kHostSets] = {&hp.start, &hp.end_in, &hp.end_comp, &hp.end_out};
    for (int i = 0; i < kHostSets; ++i) {
        events[4 + 3 * i] = &hp.in_done[i];
        events[5 + 3 * i] = &hp.comp_done[i];
        events[6 + 3 * i] = &hp.out_done[i];
    }
    cudaError_t e = cudaSuccess;
    const char* what = nullptr;
    for (cudaStream_t* st : streams) {
        if (e != cudaSuccess) break;
        e = cudaStreamCreateWithFlags(st, cudaStreamNonBlocking);
        if (e != cudaSuccess) { *st = nullptr; what = "cudaStreamCreateWithFlags"; }
    }
    for (cudaEvent_t* ev : events) {
        if (e != cudaSuccess) break;
        e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
        if (e != cudaSuccess) { *ev = nullptr; what = "cudaEventCreateWithFlags"; }
    }
    if (e != cudaSuccess) {
        for (cudaEvent_t* ev : events) if (*ev) { cudaEventDestroy(*ev); *ev = nullptr; }
        for (cudaStream_t* st : streams) if (*st) { cudaStreamDestroy(*st); *st = nullptr; }
        return cuda_fail(what, e);
    }
    hp.ready = true;
    return 0;
}

// Heads per pipeline stage: the caller's choice; else about ten stages where the kernel takes about as long as the
// copies or longer (the first group's copy-in and the last group's copy-out are not overlapped with anything, so
// short stages pay), and about five where the copies set the pace (their rows get longer, which the copy engines
// like: measured 16.4 against 18.6 ms on the 512-key cross-attention shape); copy rows of at least 512 bytes.
int host_heads_per_stage(int B, int H, int Lq, int Lk, int D, unsigned flags, int requested) {
    if (requested > 0) return requested < H ? requested : H;
    const bool fwd_only = (flags & ATTN_JVP_FWD_ONLY) != 0;
    const bool jvp_kv = !fwd_only && (flags & ATTN_JVP_KV_TANGENT_FREE) == 0;
    const double cells = (double)B * H * (double)Lq * (double)Lk * D;
    const double t_kernel = (fwd_only ? 4.0 : (jvp_kv ? 12.0 : 8.0)) * cells / 1.3e15;           // seconds, roughly
    const double bytes_in = 2.0 * D * B * H * ((fwd_only ? 1.0 : 2.0) * Lq + (jvp_kv ? 4.0 : 2.0) * Lk);
    const double t_copy = bytes_in / 45e9;
    const int stages = (t_kernel > 0.8 * t_copy) ? 10 : 5;
    int hg = (H + stages - 1) / stages;
    const int min_heads = (512 + D * 2 - 1) / (D * 2);
    if (hg < min_heads) hg = min_heads;
    return hg < H ? hg : H;
}

struct HostLayout {
    size_t nq, nk, nl;     // bytes of one Q-side tensor, one K-side tensor, the LSE block of a head group (padded)
    size_t set_bytes;      // one buffer set: q, tq, o, to, k, v, tk, tv, lse
    size_t total;          // kHostSets sets
};
HostLayout host_layout(int B, int Lq, int Lk, int D, int hg) {
    auto pad = [](size_t n) { return (n + 255) & ~(size_t)255; };
    HostLayout L;
    L.nq = pad((size_t)B * Lq * hg * D * 2);
    L.nk = pad((size_t)B * Lk * hg * D * 2);
    L.nl = pad((size_t)B * hg * Lq * 4);
    L.set_bytes = 4 * L.nq + 4 * L.nk + L.nl;
    L.total = kHostSets * L.set_bytes;
    return L;
}

int run_host(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv, void* o,
             void* to, float* lse, int B, int H, int Lq, int Lk, int D, float scale, unsigned flags,
             int heads_per_stage, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    if (flags & ~(ATTN_JVP_KV_TANGENT_FREE | ATTN_JVP_FWD_ONLY)) return ATTN_JVP_ERR_FLAGS;
    const bool fwd_only = (flags & ATTN_JVP_FWD_ONLY) != 0;
    const bool jvp_kv = !fwd_only && (flags & ATTN_JVP_KV_TANGENT_FREE) == 0;
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || heads_per_stage < 0) return ATTN_JVP_ERR_SHAPE;
    if (D != 64 && D != 128) return ATTN_JVP_ERR_UNSUPPORTED_D;
    const long double nq_all = (long double)B * H * Lq * D, nk_all = (long double)B * H * Lk * D;
    if (nq_all * 2 > 9.0e18L || nk_all * 2 > 9.0e18L) return ATTN_JVP_ERR_SHAPE;
    if (!q || !k || !v || !o || !lse || !workspace) return ATTN_JVP_ERR_NULL;
    if (!fwd_only && (!tq || !to)) return ATTN_JVP_ERR_NULL;
    if (jvp_kv && (!tk || !tv)) return ATTN_JVP_ERR_NULL;
    if (!std::isfinite(scale)) return ATTN_JVP_ERR_SCALE;
    if ((uintptr_t)workspace & 255u) return ATTN_JVP_ERR_ALIGN;
    const int hg = host_heads_per_stage(B, H, Lq, Lk, D, flags, heads_per_stage);
    const HostLayout lay = host_layout(B, Lq, Lk, D, hg);
    if (workspace_bytes < lay.total) return ATTN_JVP_ERR_WORKSPACE;

    // everything that can refuse the call without touching a stream comes first: nothing is enqueued on error
    int dev = 0;
    DeviceState* stp = nullptr;
    if (int rc = current_device(&dev, &stp)) return rc;
    if (int rc = get_encode_fn()) return rc;
    if (int rc = ensure_status_word(*stp)) return rc;
    HostPipe& hp = g_host_pipe[dev];
    std::lock_guard<std::mutex> guard(hp.lock);
    if (int rc = host_pipe_setup(hp)) return rc;

    const size_t row_host = (size_t)H * D * 2;      // bytes between consecutive (b, l) rows of a host tensor
    int rc = 0;
    cudaError_t ce = cudaSuccess;
    const char* what = nullptr;
    auto check = [&](cudaError_t err, const char* w) { if (err != cudaSuccess && ce == cudaSuccess) { ce = err; what = w; } };

    // everything below runs after what the caller has already put on `stream` ...
    cudaError_t e = cudaEventRecord(hp.start, stream);
    if (e != cudaSuccess) return cuda_fail("cudaEventRecord", e);
    cudaStream_t internal[3] = {hp.in, hp.comp, hp.out};
    for (cudaStream_t st : internal) check(cudaStreamWaitEvent(st, hp.start, 0), "cudaStreamWaitEvent");

    // The first group's copy-in and the last group's copy-out overlap with nothing: with enough groups the first one
    // is half as long, which (for a head count that is a multiple of the group length) leaves a short one at the
    // end as well.
    const int first_hc = (hg >= 2 && H >= 4 * hg) ? hg / 2 : hg;
    int h0 = 0;
    for (int g = 0; h0 < H && rc == 0 && ce == cudaSuccess; ++g) {
        const int set = g % kHostSets;
        const int want = (g == 0) ? first_hc : hg;
        const int hc = (H - h0 < want) ? H - h0 : want;
        char* base = static_cast<char*>(workspace) + (size_t)set * lay.set_bytes;
        char* d_q = base;
        char* d_tq = d_q + lay.nq;
        char* d_o = d_tq + lay.nq;
        char* d_to = d_o + lay.nq;
        char* d_k = d_to + lay.nq;
        char* d_v = d_k + lay.nk;
        char* d_tk = d_v + lay.nk;
        char* d_tv = d_tk + lay.nk;
        float* d_lse = reinterpret_cast<float*>(d_tv + lay.nk);
        const size_t row_dev = (size_t)hc * D * 2;  // the device copy of a head group is dense: [B][L][hc][D]
        const size_t head_off = (size_t)h0 * D * 2;

        // inputs of this group: gather the group's heads out of the interleaved host rows
        if (g >= kHostSets) check(cudaStreamWaitEvent(hp.in, hp.out_done[set], 0), "cudaStreamWaitEvent");
        auto h2d = [&](char* dst, const void* src, int L) {
            check(cudaMemcpy2DAsync(dst, row_dev, static_cast<const char*>(src) + head_off, row_host, row_dev,
                                    (size_t)B * L, cudaMemcpyHostToDevice, hp.in), "cudaMemcpy2DAsync (host to device)");
        };
        h2d(d_k, k, Lk);
        h2d(d_q, q, Lq);
        if (!fwd_only) h2d(d_tq, tq, Lq);
        if (jvp_kv) h2d(d_tk, tk, Lk);
        h2d(d_v, v, Lk);
        if (jvp_kv) h2d(d_tv, tv, Lk);
        check(cudaEventRecord(hp.in_done[set], hp.in), "cudaEventRecord");
        if (ce != cudaSuccess) break;

        // the kernel on the dense group (H = hc)
        check(cudaStreamWaitEvent(hp.comp, hp.in_done[set], 0), "cudaStreamWaitEvent");
        if (ce != cudaSuccess) break;
        rc = run(d_q, d_k, d_v, fwd_only ? nullptr : d_tq, jvp_kv ? d_tk : nullptr, jvp_kv ? d_tv : nullptr, d_o,
                 fwd_only ? nullptr : d_to, d_lse, nullptr, B, hc, Lq, Lk, D, scale, flags, 1, nullptr, 0, hp.comp);
        if (rc != 0) break;
        check(cudaEventRecord(hp.comp_done[set], hp.comp), "cudaEventRecord");

        // outputs of this group: scatter the heads back into the host rows; LSE is [B][H][Lq] on the host
        check(cudaStreamWaitEvent(hp.out, hp.comp_done[set], 0), "cudaStreamWaitEvent");
        check(cudaMemcpy2DAsync(static_cast<char*>(o) + head_off, row_host, d_o, row_dev, row_dev, (size_t)B * Lq,
                                cudaMemcpyDeviceToHost, hp.out), "cudaMemcpy2DAsync (device to host)");
        if (!fwd_only)
            check(cudaMemcpy2DAsync(static_cast<char*>(to) + head_off, row_host, d_to, row_dev, row_dev,
                                    (size_t)B * Lq, cudaMemcpyDeviceToHost, hp.out), "cudaMemcpy2DAsync (device to host)");
        check(cudaMemcpy2DAsync(lse + (size_t)h0 * Lq, (size_t)H * Lq * 4, d_lse, (size_t)hc * Lq * 4,
                                (size_t)hc * Lq * 4, (size_t)B, cudaMemcpyDeviceToHost, hp.out),
              "cudaMemcpy2DAsync (LSE)");
        check(cudaEventRecord(hp.out_done[set], hp.out), "cudaEventRecord");
        h0 += hc;
    }
    // ... and the caller's stream continues after all of it (also when an error cut the loop short: the internal
    // streams are never left chained to the caller's stream without the closing join)
    check(cudaEventRecord(hp.end_in, hp.in), "cudaEventRecord");
    check(cudaEventRecord(hp.end_comp, hp.comp), "cudaEventRecord");
    check(cudaEventRecord(hp.end_out, hp.out), "cudaEventRecord");
    check(cudaStreamWaitEvent(stream, hp.end_in, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(stream, hp.end_comp, 0), "cudaStreamWaitEvent");
    check(cudaStreamWaitEvent(stream, hp.end_out, 0), "cudaStreamWaitEvent");
    if (rc != 0) return rc;
    if (ce != cudaSuccess) return cuda_fail(what, ce);
    return 0;
}

}  // namespace

extern "C" {

int attn_jvp_fwd(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
                 void* o, void* to, float* lse, int B, int H, int Lq, int Lk, int D, float scale, unsigned flags) {
    return run(q, k, v, tq, tk, tv, o, to, lse, nullptr, B, H, Lq, Lk, D, scale, flags, 1, nullptr, 0, tl_stream);
}

int attn_jvp_fwd_stream(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
                        void* o, void* to, float* lse, int B, int H, int Lq, int Lk, int D, float scale,
                        unsigned flags, void* cuda_stream) {
    return run(q, k, v, tq, tk, tv, o, to, lse, nullptr, B, H, Lq, Lk, D, scale, flags, 1, nullptr, 0,
               static_cast<cudaStream_t>(cuda_stream));
}

int attn_jvp_fwd_mu(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
                    void* o, void* to, float* lse, float* mu, int B, int H, int Lq, int Lk, int D, float scale,
                    unsigned flags, void* cuda_stream) {
    if (!mu) return ATTN_JVP_ERR_NULL;
    return run(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, 1, nullptr, 0,
               static_cast<cudaStream_t>(cuda_stream));
}

size_t attn_jvp_splitkv_workspace_bytes(int B, int H, int Lq, int Lk, int D, int splits) {
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || (D != 64 && D != 128) || splits < 1) return 0;
    int tps = 0, eff = 1;
    split_plan(Lk, splits, &tps, &eff);
    if (eff <= 1) return 0;
    return split_layout(B, H, Lq, D, eff).total;
}

int attn_jvp_suggest_splits(int B, int H, int Lq, int Lk, int D) {
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || (D != 64 && D != 128)) return 1;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        (void)cudaGetLastError();
        return 1;
    }
    // Work items without a split; with at least ~60 % of the SMs busy a split only adds the merge.
    const long long items = (long long)((Lq + attn_jvp::kBlockM - 1) / attn_jvp::kBlockM) * H * B;
    if (items * 5 >= (long long)sms * 3) return 1;
    // Otherwise: the largest number of chunks that still fits one wave of CTAs, with at least four key tiles each.
    const int n_tiles = (Lk + attn_jvp::kBlockN - 1) / attn_jvp::kBlockN;
    long long splits = sms / items;
    if (splits > n_tiles / 4) splits = n_tiles / 4;
    if (splits > 1024) splits = 1024;
    return splits < 1 ? 1 : (int)splits;
}

int attn_jvp_fwd_splitkv(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
                         void* o, void* to, float* lse, float* mu, int B, int H, int Lq, int Lk, int D, float scale,
                         unsigned flags, int splits, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return run(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, splits, workspace, workspace_bytes,
               static_cast<cudaStream_t>(cuda_stream));
}

size_t attn_jvp_host_workspace_bytes(int B, int H, int Lq, int Lk, int D, int heads_per_stage) {
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || (D != 64 && D != 128) || heads_per_stage < 0) return 0;
    // (the default stage length depends on the flags, which this function does not get: the size covers the longer
    // of the two, five stages' worth of heads, which both flag-dependent choices fit into)
    const int hg_copy_bound = host_heads_per_stage(B, H, Lq, 1, D, ATTN_JVP_FWD_ONLY, heads_per_stage);
    const int hg_here = host_heads_per_stage(B, H, Lq, Lk, D, 0u, heads_per_stage);
    return host_layout(B, Lq, Lk, D, hg_copy_bound > hg_here ? hg_copy_bound : hg_here).total;
}

int attn_jvp_fwd_host(const void* q, const void* k, const void* v, const void* tq, const void* tk, const void* tv,
                      void* o, void* to, float* lse, int B, int H, int Lq, int Lk, int D, float scale, unsigned flags,
                      int heads_per_stage, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return run_host(q, k, v, tq, tk, tv, o, to, lse, B, H, Lq, Lk, D, scale, flags, heads_per_stage, workspace,
                    workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

// Scratch for callers that cannot allocate: lives in the library's device image, so every GPU that loads
// the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[ATTN_JVP_STATIC_SCRATCH_BYTES];

int attn_jvp_fwd_splitkv_static(const void* q, const void* k, const void* v, const void* tq, const void* tk,
                                const void* tv, void* o, void* to, float* lse, float* mu, int B, int H, int Lq, int Lk,
                                int D, float scale, unsigned flags, int splits, void* cuda_stream) {
    if (B < 1 || H < 1 || Lq < 1 || Lk < 1 || splits < 1) return ATTN_JVP_ERR_SHAPE;
    if (D != 64 && D != 128) return ATTN_JVP_ERR_UNSUPPORTED_D;
    const size_t need = attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits);
    if (need > (size_t)ATTN_JVP_STATIC_SCRATCH_BYTES) {
        snprintf(tl_cuda_msg, sizeof tl_cuda_msg, "this call needs %zu bytes of scratch, the built-in buffer holds %zu",
                 need, (size_t)ATTN_JVP_STATIC_SCRATCH_BYTES);
        return ATTN_JVP_ERR_STATIC_SCRATCH;
    }
    int dev = 0;
    DeviceState* stp = nullptr;
    if (int rc = current_device(&dev, &stp)) return rc;
    void* scratch = stp->static_scratch.load(std::memory_order_acquire);
    if (!scratch) {
        // In host code the array's name only stands for the symbol; its address on the current device has to be
        // asked for.  Done once per device, on the first call here.
        std::lock_guard<std::mutex> guard(stp->lock);
        scratch = stp->static_scratch.load(std::memory_order_relaxed);
        if (!scratch) {
            cudaError_t e = cudaGetSymbolAddress(&scratch, g_static_scratch);
            if (e != cudaSuccess) return cuda_fail("cudaGetSymbolAddress(static scratch)", e);
            stp->static_scratch.store(scratch, std::memory_order_release);
        }
    }
    return run(q, k, v, tq, tk, tv, o, to, lse, mu, B, H, Lq, Lk, D, scale, flags, splits, scratch,
               (size_t)ATTN_JVP_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream), /*may_allocate=*/false);
}

int attn_jvp_qknorm_fwd(const void* x, const void* tx, const float* w, void* y, void* ty, long long rows, int D,
                        float eps, void* cuda_stream) {
    if (rows < 1) return ATTN_JVP_ERR_SHAPE;
    if (D != 64 && D != 128) return ATTN_JVP_ERR_UNSUPPORTED_D;
    if (!x || !w || !y) return ATTN_JVP_ERR_NULL;
    if ((tx == nullptr) != (ty == nullptr)) return ATTN_JVP_ERR_NULL;     // tangent in and out go together
    if (!std::isfinite(eps) || eps < 0.0f) return ATTN_JVP_ERR_SCALE;
    const void* ptrs[5] = {x, tx, w, y, ty};
    for (const void* p : ptrs) if (p && ((uintptr_t)p & 15u)) return ATTN_JVP_ERR_ALIGN;
    const size_t bytes = (size_t)rows * D * 2;
    if (overlaps(y, bytes, x, bytes) || overlaps(y, bytes, tx, bytes) || overlaps(ty, bytes, x, bytes) ||
        overlaps(ty, bytes, tx, bytes) || overlaps(y, bytes, ty, bytes) || overlaps(y, bytes, w, (size_t)D * 4) ||
        overlaps(ty, bytes, w, (size_t)D * 4))
        return ATTN_JVP_ERR_ALIAS;
    int dev = 0;
    DeviceState* stp = nullptr;
    if (int rc = current_device(&dev, &stp)) return rc;
    const int sms = stp->sm_count;
    cudaError_t e;
    const int rows_per_block = 256 / (D / 8);
    long long blocks = (rows + rows_per_block - 1) / rows_per_block;
    const long long cap = (long long)sms * 16;                 // a multiple of the SM count; the kernel strides
    if (blocks > cap) blocks = cap;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const uint4* xp = static_cast<const uint4*>(x);
    const uint4* tp = static_cast<const uint4*>(tx);
    uint4* yp = static_cast<uint4*>(y);
    uint4* typ = static_cast<uint4*>(ty);
    if (D == 128) {
        if (tx) attn_jvp::qknorm_jvp_kernel<128, true><<<(unsigned)blocks, 256, 0, st>>>(xp, tp, w, yp, typ, rows, eps);
        else attn_jvp::qknorm_jvp_kernel<128, false><<<(unsigned)blocks, 256, 0, st>>>(xp, tp, w, yp, typ, rows, eps);
    } else {
        if (tx) attn_jvp::qknorm_jvp_kernel<64, true><<<(unsigned)blocks, 256, 0, st>>>(xp, tp, w, yp, typ, rows, eps);
        else attn_jvp::qknorm_jvp_kernel<64, false><<<(unsigned)blocks, 256, 0, st>>>(xp, tp, w, yp, typ, rows, eps);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail("qknorm kernel launch", e);
    return 0;
}

int attn_jvp_selftest_bounded_wait(void* cuda_stream) {
    int dev = 0;
    DeviceState* stp = nullptr;
    if (int rc = current_device(&dev, &stp)) return rc;
    if (int rc = ensure_status_word(*stp)) return rc;
    attn_jvp::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        stp->host_status_dev.load(std::memory_order_acquire));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail("self-test kernel launch", e);
    return 0;
}

int attn_jvp_set_tuning(int knob, int value) {
    if (knob == ATTN_JVP_TUNE_SOFTMAX_GROUPS && value >= 0 && value <= 2) {
        g_tune_softmax_groups.store(value, std::memory_order_relaxed);
        return 0;
    }
    if (knob == ATTN_JVP_TUNE_CTA_PAIR && value >= 0 && value <= 2) {
        g_tune_cta_pair.store(value, std::memory_order_relaxed);
        return 0;
    }
    return ATTN_JVP_ERR_FLAGS;
}

int attn_jvp_set_stream(void* cuda_stream) {
    tl_stream = static_cast<cudaStream_t>(cuda_stream);
    return 0;
}

int attn_jvp_device_status(void) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    DeviceState& ds = g_dev[dev];
    int st = 0;
    int* hp = ds.host_status.load(std::memory_order_acquire);
    if (hp) {
        st = *reinterpret_cast<volatile int*>(hp);
        if (st != 0) *reinterpret_cast<volatile int*>(hp) = 0;
    }
    // The kernels also raise a device-side flag (later launches test it and return at once).  Reading it is a
    // blocking copy, so it is read only when it can hold news: a timeout was just reported through the status
    // word (then it has to be cleared), or kernels ran here before the status word existed (then it is the only
    // record, which is the case when only the allocation-free entry point has been used).
    if (st != 0 || ds.unwatched_launch.load(std::memory_order_acquire)) {
        int flag = 0;
        if (cudaMemcpyFromSymbol(&flag, attn_jvp::g_abort_flag, sizeof(int)) == cudaSuccess) {
            if (flag != 0) {
                if (st == 0) st = ATTN_JVP_ERR_DEVICE_TIMEOUT;
                const int zero = 0;
                cudaMemcpyToSymbol(attn_jvp::g_abort_flag, &zero, sizeof(int));   // let later launches run again
            }
            if (hp) ds.unwatched_launch.store(false, std::memory_order_release);
        }
    }
    return st;
}

const char* attn_jvp_strerror(int code) {
    switch (code) {
        case ATTN_JVP_OK: return "ok";
        case ATTN_JVP_ERR_NULL: return "a required pointer is NULL";
        case ATTN_JVP_ERR_SHAPE: return "B, H, Lq and Lk must be >= 1 and the tensor sizes and the number of work items must not overflow";
        case ATTN_JVP_ERR_UNSUPPORTED_D: return "head dimension D must be 64 or 128";
        case ATTN_JVP_ERR_ALIGN: return "tensor pointers must be 16-byte aligned";
        case ATTN_JVP_ERR_FLAGS: return "unknown flag bits";
        case ATTN_JVP_ERR_SCALE: return "scale must be finite";
        case ATTN_JVP_ERR_ALIAS: return "an output buffer overlaps an input or another output";
        case ATTN_JVP_ERR_ARCH: return "the current device is not compute capability 10.x (sm_100a)";
        case ATTN_JVP_ERR_CUDA:
            snprintf(tl_strerror_buf, sizeof tl_strerror_buf, "CUDA call failed: %s", tl_cuda_msg);
            return tl_strerror_buf;
        case ATTN_JVP_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired; the kernel stopped early";
        case ATTN_JVP_ERR_DEVICE_LAYOUT: return "the kernel's shared-memory layout did not fit; nothing was computed";
        case ATTN_JVP_ERR_WORKSPACE: return "the workspace is smaller than the matching *_workspace_bytes() function asks for";
        case ATTN_JVP_ERR_STATIC_SCRATCH:
            snprintf(tl_strerror_buf, sizeof tl_strerror_buf, "built-in scratch too small: %s", tl_cuda_msg);
            return tl_strerror_buf;
        default: return "unknown error code";
    }
}

int attn_jvp_version(void) { return kVersion; }

// Diagnostics after ATTN_JVP_ERR_DEVICE_TIMEOUT: which wait gave up first on the current device.  out[0..3] =
// shared-memory address of the barrier, parity waited for, threadIdx.x, blockIdx.x; returns 1 if a record exists
// (and clears it), 0 if not, -1 on a CUDA error.  Blocking (copies from the device).
int attn_jvp_debug_timeout_info(unsigned* out) {
    unsigned info[5] = {};
    if (!out || cudaMemcpyFromSymbol(info, attn_jvp::g_timeout_info, sizeof info) != cudaSuccess) return -1;
    for (int i = 0; i < 4; ++i) out[i] = info[i];
    if (info[4] == 0) return 0;
    const unsigned zero[5] = {};
    cudaMemcpyToSymbol(attn_jvp::g_timeout_info, zero, sizeof zero);
    return 1;
}
#ifdef ATTN_JVP_DEBUG
int attn_jvp_debug_barrier_layout(unsigned* out, int n) {
    if (n < 14) return -1;
    return cudaMemcpyFromSymbol(out, attn_jvp::g_barrier_layout, 14 * sizeof(unsigned)) == cudaSuccess ? 14 : -1;
}
#endif

#ifdef ATTN_JVP_TRACE
// Debug builds only: copies the in-kernel timeline (clock64 stamps) of the traced CTA to `dst`.
int attn_jvp_debug_read_trace(long long* dst, int n) {
    const int total = attn_jvp::kTraceEvents * attn_jvp::kTraceSteps;
    if (n < total) return -total;
    cudaError_t e = cudaMemcpyFromSymbol(dst, attn_jvp::g_trace, sizeof(long long) * total);
    return e == cudaSuccess ? total : -1;
}
#endif

}  // extern "C"
