// C ABI of the MoDA operator (see include/moda.h): argument validation, tensor-map
// construction and kernel launches.  Everything that computes lives in the kernels.
#include "../../include/moda.h"

#include <cstdint>
#include <cstring>
#include <mutex>

#include "moda_bwd.cuh"
#include "moda_bwd_fused.cuh"
#include "moda_cache.cuh"
#include "moda_decode.cuh"
#include "moda_depth_gqa.cuh"
#include "moda_fwd.cuh"
#include "moda_fwd_wide.cuh"
#include "moda_mass.cuh"
#include "moda_kvproj.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace moda;

thread_local int tl_last_cuda_error = 0;

// One thread waits on an mbarrier that nothing arrives at; the bounded wait gives up after `limit_ns`
// and records (MODA_SELFTEST_WAIT_SITE << 8) | 1 exactly as a production kernel's wait would.
__global__ void wait_timeout_selftest_kernel(uint64_t limit_ns) {
    __shared__ __align__(8) uint64_t bar_word;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0;
        mbar_init(smem_u32(&bar_word), 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar_word), 0, &abort_word, MODA_SELFTEST_WAIT_SITE, limit_ns);
}

inline bool cuda_ok(cudaError_t e) {
    if (e == cudaSuccess) return true;
    tl_last_cuda_error = static_cast<int>(e);
    (void)cudaGetLastError();   // clear the sticky-free error so that later calls start clean
    return false;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Tensor map over a contiguous bf16 [B][T][H][d] tensor; one box = 128 positions x 64
// features of one (b, h), written to shared memory with the 128-byte swizzle.
// Out-of-range rows (ragged last tile) read as zero and are dropped on store.
bool make_bthd_map(CUtensorMap* map, const void* base, int B, int T, int H, int d, int box_rows = kTileRows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) { tl_last_cuda_error = static_cast<int>(cudaErrorNotSupported); return false; }
    const cuuint64_t dims[4] = {cuuint64_t(d), cuuint64_t(H), cuuint64_t(T), cuuint64_t(B)};
    const cuuint64_t strides[3] = {cuuint64_t(d) * 2, cuuint64_t(H) * d * 2, cuuint64_t(T) * H * d * 2};
    const cuuint32_t box[4] = {64, 1, cuuint32_t(box_rows), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { tl_last_cuda_error = static_cast<int>(cudaErrorInvalidValue); return false; }
    return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int B, int T, int H, int d) {
    if (B < 1 || T < 1 || H < 1) return MODA_ERR_BAD_SHAPE;
    if (d != 64 && d != 128) return MODA_ERR_BAD_HEAD_DIM;
    // keep every element count and grid size inside 31 / 63 bits
    const long long rows = (long long)B * H * num_tiles(T);
    if (rows > 0x3fffffffLL) return MODA_ERR_BAD_SHAPE;
    if ((long long)B * T > 0x7fffffffLL / H) return MODA_ERR_BAD_SHAPE;
    return MODA_OK;
}

// Query heads H on H_kv key/value heads: H_kv must divide H; 1 to 8, 16 or 32 heads per group.
// The softmax scale: finite and at least 1e-20.  Zero (a uniform softmax) and negative scales are not served: the
// kernels take row maxima of the raw scores and scale afterwards, masked scores are -inf times the scale, and the
// fused backward divides LSE by it.
int check_scale(float scale) {
    return (std::isfinite(scale) && scale >= 1e-20f) ? MODA_OK : MODA_ERR_BAD_SCALE;
}

int check_groups(int H, int H_kv) {
    if (H_kv < 1 || H % H_kv != 0) return MODA_ERR_BAD_GROUP;
    const int G = H / H_kv;
    if (!(G <= 8 || G == 16 || G == 32)) return MODA_ERR_BAD_GROUP;
    return MODA_OK;
}

// Host-visible mirror of the device status word, one per device: four bytes of pinned host memory that
// the device can write (zero-copy).  A kernel whose wait runs out stores its code there as well as in
// g_moda_status, so the next call on that device sees it with a plain load -- no synchronisation --
// and returns MODA_ERR_DEVICE_TIMEOUT instead of queueing work behind a failed kernel.
constexpr int kMaxDevices = 64;
std::mutex g_mirror_mutex;
volatile int* g_status_mirror[kMaxDevices] = {};

int ensure_status_mirror(int dev) {
    if (dev < 0 || dev >= kMaxDevices) return MODA_OK;         // beyond the table: moda_last_status still works
    std::lock_guard<std::mutex> lock(g_mirror_mutex);
    if (g_status_mirror[dev] != nullptr) return MODA_OK;
    int* host = nullptr;
    int* dev_alias = nullptr;
    if (!cuda_ok(cudaHostAlloc(reinterpret_cast<void**>(&host), sizeof(int), cudaHostAllocMapped))) return MODA_ERR_CUDA;
    *host = 0;
    if (!cuda_ok(cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev_alias), host, 0)) ||
        !cuda_ok(cudaMemcpyToSymbol(g_moda_status_host, &dev_alias, sizeof(dev_alias)))) {
        (void)cudaFreeHost(host);
        return MODA_ERR_CUDA;
    }
    g_status_mirror[dev] = host;
    return MODA_OK;
}

// Device check of every launching entry point: an sm_100 part, and no kernel of an earlier call on this
// device has given up a wait.  `may_allocate` = false (the entry point that must not allocate) skips the
// one-time creation of the status mirror; a mirror made by an earlier call is still consulted.
int check_device(bool may_allocate = true) {
    static thread_local int cached_dev = -1;
    static thread_local int cached_rc = MODA_ERR_DEVICE;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (dev != cached_dev) {
        int major = 0;
        if (!cuda_ok(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev))) return MODA_ERR_CUDA;
        cached_dev = dev;
        cached_rc = (major == 10) ? MODA_OK : MODA_ERR_DEVICE;
    }
    if (cached_rc != MODA_OK) return cached_rc;
    if (dev >= 0 && dev < kMaxDevices) {
        volatile int* mirror = g_status_mirror[dev];
        if (mirror == nullptr && may_allocate) {
            if (int rc = ensure_status_mirror(dev)) return rc;
            mirror = g_status_mirror[dev];
        }
        if (mirror != nullptr && *mirror != 0) return MODA_ERR_DEVICE_TIMEOUT;
    }
    return MODA_OK;
}

template <typename Kernel>
bool set_smem_limit(Kernel k, int bytes) {
    return cuda_ok(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
}

// d = 128 runs moda_fwd_kernel (one softmax warpgroup: the tensor pipe and the MMA issue rate set the
// pace); d = 64 runs moda_fwd2_kernel (two softmax warpgroups, three score buffers: the exponentials do).
// Which forward kernel at d = 128: one K stage and a five-unit depth ring when the depth stream
// outweighs the sequence work (measured: - 6 % at l d / T = 0.72, - 3 % at 0.5, slower below),
// otherwise two K stages and a three-unit ring.
inline bool fwd_depth_heavy(int T_q, int T_kv, int l, int d) {
    // against the mean number of key tiles of a query tile, (2 T_kv - T_q) / 256: with T_q = T_kv = T this is 2 l d >= T
    return d == 128 && l > 0 && 2ll * l * d >= 2ll * T_kv - T_q;
}

// Whether a grouped-query forward runs its depth part as the separate per-position kernel.  Measured at
// d = 64 (T = 16384, 8 key/value heads): the fused row-local path costs about 2.3 us per (query head per
// group, slot), the separate kernel about 200 us plus 11.7 us per slot whatever the group size, so the
// separate kernel wins for large groups with many slots (G = 8 from l = 31, G = 7 from 46, G = 6 from 96).
// At d = 128 (T = 8192) it wins only for 8 heads per group from about 45 slots (l = 64: 2.31 -> 2.08 ms;
// l = 24: 1.40 -> 1.58 ms; G = 6, l = 64: 1.74 -> 1.84 ms).
inline bool gqa_depth_split(int d, int G, int l) {
    if (d == 128) return (G == 8 || G == 16 || G == 32) && l >= 48;
    if (G == 16 || G == 32) return l >= 14;                        // 16 heads per launch (G = 16, l = 16: 0.73 -> 0.67 ms; l = 8: 0.51 -> 0.70)
    return G >= 6 && G <= 8 && l * (23 * G - 117) > 2000;
}

template <int D, int G>
int launch_depth_merge_g(const DepthMergeParams& m, cudaStream_t stream) {
    constexpr int kBytes = depth_merge_smem_bytes<D>();
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(depth_merge_fwd_kernel<D, G>, kBytes)) return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    const long long blocks = (long long)m.B * m.Hk * ((m.T + kDgPos - 1) / kDgPos);
    if (blocks > 0x7fffffffLL) return MODA_ERR_BAD_SHAPE;
    depth_merge_fwd_kernel<D, G><<<unsigned(blocks), kDgThreads, kBytes, stream>>>(m);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}
template <int D>
int launch_depth_merge(DepthMergeParams m, cudaStream_t stream) {
    const int G = m.H / m.Hk;
    m.h0 = 0;
    switch (G) {
        case 2: return launch_depth_merge_g<D, 2>(m, stream);
        case 3: return launch_depth_merge_g<D, 3>(m, stream);
        case 4: return launch_depth_merge_g<D, 4>(m, stream);
        case 5: return launch_depth_merge_g<D, 5>(m, stream);
        case 6: return launch_depth_merge_g<D, 6>(m, stream);
        case 7: return launch_depth_merge_g<D, 7>(m, stream);
        case 8: return launch_depth_merge_g<D, 8>(m, stream);
        case 16: return launch_depth_merge_g<D, 16>(m, stream);       // 16 heads fill the 16 rows of the warp-level products
        case 32:
            for (m.h0 = 0; m.h0 < G; m.h0 += 16)
                if (int rc = launch_depth_merge_g<D, 16>(m, stream)) return rc;
            return MODA_OK;
        default: return MODA_ERR_BAD_GROUP;
    }
}

// How the depth cache of a call is laid out: row-interleaved bf16 (the default), e4m3 codes with row scales, or
// position-major bf16 (moda_cache.cuh).
enum CacheKind { kCacheRows = 0, kCacheE4m3 = 1, kCachePm = 2 };

// Dynamic shared memory of the forward kernel that reads an e4m3 depth cache (only the variant each head size runs exists).
template <int D>
constexpr int fwd_smem_e4m3() {
    if constexpr (D == 64) return Fwd2Smem<64, true>::kDynamic;
    else return FwdSmem<128, 2, true>::kDynamic;
}

template <int D>
int launch_fwd(const void* Q, const void* K, const void* V, const void* depth_kv, int B, int T, int T_kv, int H, int Hk, int l,
               float scale, void* O, float* LSE, void* append_slot, cudaStream_t stream, CacheKind kind = kCacheRows) {
    const bool fp8 = kind == kCacheE4m3, pm = kind == kCachePm;
    constexpr bool kWide = (D == 64);
    constexpr int kSmem = kWide ? Fwd2Smem<D>::kDynamic : FwdSmem<D, 2>::kDynamic;
    constexpr int kSmem8 = fwd_smem_e4m3<D>();
    constexpr int kSmemDeep = FwdSmem<128, 1>::kDynamic;
    constexpr int kThreads = kWide ? kFwd2Threads : kFwdThreads;
    CUtensorMap mQ, mK, mV, mO;
    if (!make_bthd_map(&mQ, Q, B, T, H, D) || !make_bthd_map(&mK, K, B, T_kv, Hk, D) ||
        !make_bthd_map(&mV, V, B, T_kv, Hk, D) || !make_bthd_map(&mO, O, B, T, H, D))
        return MODA_ERR_CUDA;
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        bool ok;
        if constexpr (kWide) ok = set_smem_limit(moda_fwd2_kernel<D>, kSmem) && set_smem_limit(moda_fwd2_kernel<D, true>, kSmem8);
        else ok = set_smem_limit(moda_fwd_kernel<D, 2>, kSmem) && set_smem_limit(moda_fwd_kernel<128, 1>, kSmemDeep) &&
                  set_smem_limit(moda_fwd_kernel<128, 2, true>, kSmem8);
        if (!ok) return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    FwdParams p;
    p.Q = static_cast<const __nv_bfloat16*>(Q);
    p.K = static_cast<const __nv_bfloat16*>(K);
    p.V = static_cast<const __nv_bfloat16*>(V);
    p.depth_kv = depth_kv;
    p.O = static_cast<__nv_bfloat16*>(O);
    p.LSE = LSE;
    p.B = B; p.T = T; p.H = H; p.l = l;
    p.T_kv = T_kv; p.kv_off = T_kv - T;
    p.G = H / Hk;
    p.scale_log2 = scale * kLog2e;
    p.append_slot = append_slot;
    // The d = 128 kernel takes a pair of query tiles per CTA when the call is causal over equally many keys and queries
    // (the pairs then have equal work) and the equal-sized CTAs fill their last wave (at least 93 % of the SM slots of
    // all waves; 512 pairs on 148 SMs would idle a seventh of them, measured + 4 % at c3 with B = 1), or when the depth
    // stream outweighs the sequence work anyway (c2: - 5 %).  Otherwise, and at d = 64, one tile per CTA, heaviest first (a
    // prefill's tiles are nearly equal already and halving the CTA count costs a wave: + 15 % measured).
    const long long n_pairs = (long long)B * H * num_tile_pairs(num_tiles(T));
    const long long pair_waves = (n_pairs + 147) / 148;
    const bool pair = !kWide && T_kv == T && n_pairs >= 2 * 148 &&
                      (100 * n_pairs >= 93 * 148 * pair_waves || fwd_depth_heavy(T, T_kv, l, D));
    p.pair = pair ? 1 : 0;
    const unsigned grid = unsigned(B) * H * (pair ? num_tile_pairs(num_tiles(T)) : num_tiles(T));
    // Grouped-query calls: the sequence kernel runs without depth slots and a second kernel adds the depth
    // part of all heads of a group at once (moda_depth_gqa.cuh).
    // An e4m3 cache is always read by the row-local depth warps of the sequence kernel.
    // A position-major cache is always read by the per-position kernel.
    const bool split_depth = pm ? l > 0 : (!fp8 && gqa_depth_split(D, p.G, l));
    if (split_depth) p.l = 0;
    if (fp8) {
        if constexpr (kWide) moda_fwd2_kernel<D, true><<<grid, kThreads, kSmem8, stream>>>(mQ, mK, mV, mO, p);
        else moda_fwd_kernel<128, 2, true><<<grid, kThreads, kSmem8, stream>>>(mQ, mK, mV, mO, p);
    } else if (kWide) moda_fwd2_kernel<D><<<grid, kThreads, kSmem, stream>>>(mQ, mK, mV, mO, p);
    else if (!split_depth && fwd_depth_heavy(T, T_kv, l, D)) moda_fwd_kernel<128, 1><<<grid, kThreads, kSmemDeep, stream>>>(mQ, mK, mV, mO, p);
    else moda_fwd_kernel<D, 2><<<grid, kThreads, kSmem, stream>>>(mQ, mK, mV, mO, p);
    if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    if (split_depth) {
        DepthMergeParams m;
        m.Q = static_cast<const __nv_bfloat16*>(Q);
        m.depth_kv = static_cast<const __nv_bfloat16*>(depth_kv);
        m.O = static_cast<__nv_bfloat16*>(O);
        m.LSE = LSE;
        m.B = B; m.T = T; m.H = H; m.Hk = Hk; m.l = l;
        m.scale_log2 = scale * kLog2e;
        m.pm = pm ? 1 : 0;
        if (int rc = launch_depth_merge<D>(m, stream)) return rc;
    }
    return MODA_OK;
}

// Which dQ kernel at d = 128: two K/V stages and a five-unit depth ring when streaming the depth cache
// outweighs the sequence contractions (measured cross-over near l d / T = 0.6), otherwise three K/V
// stages and a three-unit ring.  At d = 64 three K/V stages and eight units fit together.
inline bool dq_depth_heavy(int T, int l, int d) {
    return d == 128 && l > 0 && 3ll * l * d >= 2ll * T;
}

// Whether a grouped-query backward runs its depth part as the separate per-position kernel (and with it the fused form
// of the sequence part): always.  Measured (8 key/value heads; d = 64 at T = 16384, d = 128 at T = 8192; ms, row-local
// path with the split sequence kernels -> fused sequence kernel + per-position kernel): G = 2, l = 4: 2.76 -> 1.91;
// G = 4, l = 16: 6.10 -> 3.76; G = 8, l = 8: 11.26 -> 7.38; G = 16, l = 4: 21.8 -> 15.0; d = 128, G = 2, l = 4: 1.03 -> 1.05
// (the only tie).  The row-local path remains what MODA_BWD_DETERMINISTIC selects.
inline bool gqa_depth_split_bwd(int d, int G, int l) {
    (void)d;
    return l > 0 && G >= 2;
}

template <int D, int G>
int launch_depth_bwd_g(const DepthBwdParams& m, cudaStream_t stream) {
    constexpr int kBytes = DepthBwdSmem<D, G>::kTotal;
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(depth_bwd_gqa_kernel<D, G>, kBytes)) return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    const long long blocks = (long long)m.B * m.Hk * num_tiles(m.T) * (kTileRows / db_pos<D>());
    if (blocks > 0x7fffffffLL) return MODA_ERR_BAD_SHAPE;
    depth_bwd_gqa_kernel<D, G><<<unsigned(blocks), db_pos<D>() * 32, kBytes, stream>>>(m);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}
template <int D>
int launch_depth_bwd(DepthBwdParams m, cudaStream_t stream) {
    const int G = m.H / m.Hk;
    m.h0 = 0;
    switch (G) {
        case 2: return launch_depth_bwd_g<D, 2>(m, stream);
        case 3: return launch_depth_bwd_g<D, 3>(m, stream);
        case 4: return launch_depth_bwd_g<D, 4>(m, stream);
        case 5: return launch_depth_bwd_g<D, 5>(m, stream);
        case 6: return launch_depth_bwd_g<D, 6>(m, stream);
        case 7: return launch_depth_bwd_g<D, 7>(m, stream);
        case 8: return launch_depth_bwd_g<D, 8>(m, stream);
        case 16: return launch_depth_bwd_g<D, 16>(m, stream);      // 16 heads fill the 16 rows (or the 16-deep contraction)
        case 32:
            for (m.h0 = 0; m.h0 < G; m.h0 += 16) {
                if (int rc = launch_depth_bwd_g<D, 16>(m, stream)) return rc;
                m.accumulate = 1;                                   // the second group of 16 adds to the first one's gradients
            }
            return MODA_OK;
        default: return MODA_ERR_BAD_GROUP;
    }
}

// Which form of the backward a call takes: the fused form (moda_bwd_fused.cuh) unless the caller asks for
// reproducible bits.  Grouped-query calls in the fused form run their depth part as the per-position kernel; in
// the split form they stay row-local: its dQ pass leaves the per-row factors that depth_grad_group_kernel sums
// over the heads of a group.
inline bool bwd_uses_fused(int d, int G, int l, bool deterministic) {
    if (deterministic) return false;
    return G == 1 || l == 0 || gqa_depth_split_bwd(d, G, l);
}

template <int D>
int launch_bwd_fused(const BwdArgs& a, int stages, cudaStream_t stream) {
    const int B = a.B, T = a.T, H = a.H, Hk = a.Hk, G = a.H / a.Hk;
    using L = FusedSmem<D>;
    CUtensorMap mK, mV, mQ, mdO, mdK, mdV;
    if (!make_bthd_map(&mK, a.K, B, T, Hk, D) || !make_bthd_map(&mV, a.V, B, T, Hk, D) ||
        !make_bthd_map(&mQ, a.Q, B, T, H, D) || !make_bthd_map(&mdO, a.dO, B, T, H, D) ||
        !make_bthd_map(&mdK, a.dK, B, T, Hk, D) || !make_bthd_map(&mdV, a.dV, B, T, Hk, D))
        return MODA_ERR_CUDA;
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(moda_bwd_fused_kernel<D>, L::kDynamic)) return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    float* delta = static_cast<float*>(a.workspace);
    float* dq_acc = reinterpret_cast<float*>(static_cast<char*>(a.workspace) + bwd_fused_rowterm_bytes(B, T, H));
    const bool split_depth = G > 1 && a.l > 0;             // depth part by the per-position kernel after the finish kernel
    const unsigned tiles = unsigned(B) * H * num_tiles(T);
    constexpr int kRowThreads = kTileRows * (D / 32);
    if (stages & 1) {
        RowsParams r;
        r.Q = static_cast<const __nv_bfloat16*>(a.Q);
        r.O = static_cast<const __nv_bfloat16*>(a.O);
        r.dO = static_cast<const __nv_bfloat16*>(a.dO);
        r.depth_kv = a.depth_kv;
        r.d_depth_kv = static_cast<__nv_bfloat16*>(a.d_depth_kv);
        r.LSE = a.LSE; r.delta = delta; r.dq_acc = dq_acc;
        r.B = B; r.T = T; r.H = H; r.l = split_depth ? 0 : a.l;
        r.accumulate = a.accumulate_depth ? 1 : 0;
        r.scale = a.scale; r.scale_log2 = a.scale * kLog2e;
        if (a.fp8_cache) bwd_rows_kernel<D, true><<<tiles, kRowThreads, 0, stream>>>(r);
        else bwd_rows_kernel<D><<<tiles, kRowThreads, 0, stream>>>(r);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    }
    if (stages & 2) {
        FusedParams f;
        f.LSE = a.LSE; f.delta = delta; f.dq_acc = dq_acc;
        f.B = B; f.T = T; f.H = H; f.G = G;
        f.scale = a.scale; f.scale_log2 = a.scale * kLog2e;
        const unsigned grid = unsigned(B) * Hk * num_tiles(T);
        moda_bwd_fused_kernel<D><<<grid, L::kThreads, L::kDynamic, stream>>>(mK, mV, mQ, mdO, mdK, mdV, f);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    }
    if (stages & 4) {
        bwd_dq_finish_kernel<D><<<tiles, kRowThreads, 0, stream>>>(dq_acc, static_cast<__nv_bfloat16*>(a.dQ), B, T, H, a.scale);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
        if (split_depth) {
            DepthBwdParams m;
            m.Q = static_cast<const __nv_bfloat16*>(a.Q);
            m.dO = static_cast<const __nv_bfloat16*>(a.dO);
            m.depth_kv = static_cast<const __nv_bfloat16*>(a.depth_kv);
            m.d_depth_kv = static_cast<__nv_bfloat16*>(a.d_depth_kv);
            m.dQ = static_cast<__nv_bfloat16*>(a.dQ);
            m.LSE = a.LSE; m.delta = delta;
            m.B = B; m.T = T; m.H = H; m.Hk = Hk; m.l = a.l;
            m.scale = a.scale; m.scale_log2 = a.scale * kLog2e;
            m.accumulate = a.accumulate_depth ? 1 : 0;
            m.pm = a.pm_cache ? 1 : 0;
            if (int rc = launch_depth_bwd<D>(m, stream)) return rc;
        }
    }
    return MODA_OK;
}

template <int D>
int launch_bwd(const BwdArgs& a, int stages, cudaStream_t stream) {
    const int B = a.B, T = a.T, H = a.H, Hk = a.Hk, G = a.H / a.Hk;
    if (bwd_uses_fused(D, G, a.l, a.deterministic)) return launch_bwd_fused<D>(a, stages, stream);
    CUtensorMap mQ, mdO, mK64, mV64, mdQ, mK, mV, mQ64, mdO64, mdK, mdV;
    if (!make_bthd_map(&mQ, a.Q, B, T, H, D) || !make_bthd_map(&mdO, a.dO, B, T, H, D) ||
        !make_bthd_map(&mK64, a.K, B, T, Hk, D, kKeyTile) || !make_bthd_map(&mV64, a.V, B, T, Hk, D, kKeyTile) ||
        !make_bthd_map(&mdQ, a.dQ, B, T, H, D) || !make_bthd_map(&mK, a.K, B, T, Hk, D) ||
        !make_bthd_map(&mV, a.V, B, T, Hk, D) || !make_bthd_map(&mQ64, a.Q, B, T, H, D, kKeyTile) ||
        !make_bthd_map(&mdO64, a.dO, B, T, H, D, kKeyTile) || !make_bthd_map(&mdK, a.dK, B, T, Hk, D) ||
        !make_bthd_map(&mdV, a.dV, B, T, Hk, D))
        return MODA_ERR_CUDA;
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(moda_bwd_dq_kernel<D, 3>, DqSmem<D, 3>::kDynamic) ||
            (D == 128 && !set_smem_limit(moda_bwd_dq_kernel<128, 2>, DqSmem<128, 2>::kDynamic)) ||
            !set_smem_limit(moda_bwd_dkdv_kernel<D>, DkvSmem<D>::kDynamic))
            return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    float* delta = static_cast<float*>(a.workspace);
    if (stages & 1) {
        constexpr int rows_per_block = 256 / (D / 8);
        const long long nrows = (long long)B * T * H;
        const unsigned grid = unsigned((nrows + rows_per_block - 1) / rows_per_block);
        bwd_delta_kernel<D><<<grid, 256, 0, stream>>>(static_cast<const uint4*>(a.O), static_cast<const uint4*>(a.dO), delta, B, T, H);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    }
    if (stages & 2) {
        // one CTA per (batch, query head, 128-row tile)
        const unsigned grid = unsigned(B) * H * num_tiles(T);
        DqParams p;
        p.depth_kv = static_cast<const __nv_bfloat16*>(a.depth_kv);
        p.d_depth_kv = static_cast<__nv_bfloat16*>(a.d_depth_kv);
        p.LSE = a.LSE; p.delta = delta;
        const bool split_depth = gqa_depth_split_bwd(D, G, a.l);   // depth gradients by the per-position kernel below
        p.B = B; p.T = T; p.H = H; p.l = split_depth ? 0 : a.l; p.G = G;
        p.accumulate = a.accumulate_depth ? 1 : 0;
        p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
        // Grouped-query: the dQ kernel leaves R_i, dU_i per (row, slot, head) behind the row terms D_t
        // and a second, write-bound kernel forms the depth gradients as sums over each group.
        float* rowterms = reinterpret_cast<float*>(static_cast<char*>(a.workspace) + bwd_workspace_bytes(B, T, H));
        p.depth_rowterms = (G > 1 && a.l > 0 && !split_depth) ? rowterms : nullptr;
        if (dq_depth_heavy(T, p.l, D))
            moda_bwd_dq_kernel<128, 2><<<grid, kBwdDqThreads, DqSmem<128, 2>::kDynamic, stream>>>(mQ, mdO, mK64, mV64, mdQ, p);
        else
            moda_bwd_dq_kernel<D, 3><<<grid, kBwdDqThreads, DqSmem<D, 3>::kDynamic, stream>>>(mQ, mdO, mK64, mV64, mdQ, p);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
        if (split_depth) {
            DepthBwdParams m;
            m.Q = static_cast<const __nv_bfloat16*>(a.Q);
            m.dO = static_cast<const __nv_bfloat16*>(a.dO);
            m.depth_kv = static_cast<const __nv_bfloat16*>(a.depth_kv);
            m.d_depth_kv = static_cast<__nv_bfloat16*>(a.d_depth_kv);
            m.dQ = static_cast<__nv_bfloat16*>(a.dQ);
            m.LSE = a.LSE; m.delta = delta;
            m.B = B; m.T = T; m.H = H; m.Hk = Hk; m.l = a.l;
            m.scale = a.scale; m.scale_log2 = a.scale * kLog2e;
            m.accumulate = a.accumulate_depth ? 1 : 0;
            m.pm = 0;
            if (int rc = launch_depth_bwd<D>(m, stream)) return rc;
        } else if (G > 1 && a.l > 0) {
            const unsigned tiles2 = unsigned(B) * Hk * num_tiles(T) * 2;            // x {dKd, dVd}
            const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(a.Q);
            const __nv_bfloat16* go = static_cast<const __nv_bfloat16*>(a.dO);
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.d_depth_kv);
#define MODA_GROUP_CASE(GG) \
            case GG: depth_grad_group_kernel<D, GG><<<tiles2 * (D / GroupGrad<GG>::kFW / 4), kGroupGradThreads, 0, stream>>>( \
                         q, go, rowterms, out, B, T, Hk, a.l, a.scale, a.accumulate_depth ? 1 : 0); break;
            switch (G) {
                MODA_GROUP_CASE(2) MODA_GROUP_CASE(3) MODA_GROUP_CASE(4) MODA_GROUP_CASE(5)
                MODA_GROUP_CASE(6) MODA_GROUP_CASE(7) MODA_GROUP_CASE(8) MODA_GROUP_CASE(16) MODA_GROUP_CASE(32)
                default: return MODA_ERR_BAD_GROUP;
            }
#undef MODA_GROUP_CASE
            if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
        }
    }
    // dK, dV: one CTA per (batch, key/value head, 128-row tile)
    const unsigned grid = unsigned(B) * Hk * num_tiles(T);
    if (stages & 4) {
        DkvParams p;
        p.LSE = a.LSE; p.delta = delta;
        p.B = B; p.T = T; p.H = H; p.G = G;
        p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
        moda_bwd_dkdv_kernel<D><<<grid, kBwdDkvThreads, DkvSmem<D>::kDynamic, stream>>>(mK, mV, mQ64, mdO64, mdK, mdV, p);
        if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    }
    return MODA_OK;
}

template <int D, bool kToCache>
int launch_cache_copy(void* cache, int B, int T, int H, int slot, void* Xk, void* Xv, cudaStream_t stream) {
    uint4* slot_base = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(cache) + size_t(slot) * cache_slot_elems(B, T, H, D));
    const unsigned grid = unsigned(B) * H * num_tiles(T) * 2;
    depth_cache_copy_kernel<D, kToCache><<<grid, 256, 0, stream>>>(slot_base, static_cast<uint4*>(Xk), static_cast<uint4*>(Xv), T, H);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}

template <int D, bool kToCache>
int launch_cache_pm_copy(void* cache, int B, int T, int H, int slot, void* Xk, void* Xv, cudaStream_t stream) {
    uint4* slot_base = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(cache) + size_t(slot) * cache_slot_elems(B, T, H, D));
    const size_t pieces = cache_slot_elems(B, T, H, D) / 8;
    const unsigned grid = unsigned(std::min<size_t>((pieces + 255) / 256, 148 * 32));
    depth_cache_pm_copy_kernel<D, kToCache><<<grid, 256, 0, stream>>>(slot_base, static_cast<uint4*>(Xk), static_cast<uint4*>(Xv), B, T, H);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}

// Key / value projection with the write step in its epilogue: a persistent kernel on CTA pairs (clusters of two CTAs).
template <int D, int NH, bool FP8 = false>
int launch_kv_project(const void* X, const void* Wk, const void* Wv, int B, int T, int Dm, int Hk,
                      void* K_out, void* V_out, void* slot, cudaStream_t stream) {
    using L = KvProjSmem<D, NH>;
    CUtensorMap mX, mWk, mWv, mK, mV;
    if (!make_bthd_map(&mX, X, B, T, Dm / 64, 64) || !make_bthd_map(&mWk, Wk, 1, Hk * D, Dm / 64, 64, D * NH) ||
        !make_bthd_map(&mWv, Wv, 1, Hk * D, Dm / 64, 64, D * NH))
        return MODA_ERR_CUDA;
    if (!make_bthd_map(&mK, K_out ? K_out : X, B, T, K_out ? Hk : Dm / 64, K_out ? D : 64) ||
        !make_bthd_map(&mV, V_out ? V_out : X, B, T, V_out ? Hk : Dm / 64, V_out ? D : 64))
        return MODA_ERR_CUDA;
    KvProjParams p;
    p.slot = slot;
    p.B = B; p.T = T; p.Hk = Hk; p.Dm = Dm;
    p.store_kv = K_out != nullptr ? 1 : 0;
    const long long items = (long long)B * ((num_tiles(T) + 1) / 2) * (Hk / NH);
    if (items > 0x3fffffffLL) return MODA_ERR_BAD_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kProjThreads, 1, 1);
    cfg.dynamicSmemBytes = L::kDynamic;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // persistent: as many pairs as the device can hold at once (a pair needs two SMs of one cluster domain; 74 on a B200)
    static thread_local int configured_dev = -1;
    static thread_local int resident_pairs = 0;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(moda_kv_project_kernel<D, NH, FP8>, L::kDynamic)) return MODA_ERR_CUDA;
        int n = 0;
        cfg.gridDim = dim3(1024, 1, 1);                        // any multiple of the cluster size: the query asks what fits
        if (!cuda_ok(cudaOccupancyMaxActiveClusters(&n, moda_kv_project_kernel<D, NH, FP8>, &cfg)) || n < 1) return MODA_ERR_CUDA;
        resident_pairs = n;
        configured_dev = dev;
    }
    const long long clusters = items < resident_pairs ? items : resident_pairs;
    cfg.gridDim = dim3(unsigned(2 * clusters), 1, 1);
    return cuda_ok(cudaLaunchKernelEx(&cfg, moda_kv_project_kernel<D, NH, FP8>, mX, mWk, mWv, mK, mV, p)) ? MODA_OK : MODA_ERR_CUDA;
}

// Decode step: a split kernel over the KV cache and a merge kernel that adds the depth pairs.
template <int D, int G>
int launch_decode_g(const DecodeParams& p, cudaStream_t stream) {
    using L = DecodeSmem<D, G>;
    CUtensorMap mK, mV;
    // contiguous cache: [B][T_cap][Hk][d]; paged cache: [num_pages][page_size][Hk][d] (p.T_cap holds num_pages then)
    const int outer = p.block_table ? p.T_cap : p.B, rows = p.block_table ? p.page_size : p.T_cap;
    if (!make_bthd_map(&mK, p.K, outer, rows, p.Hk / p.kv_rep, D, kDecodeStageKeys) ||
        !make_bthd_map(&mV, p.V, outer, rows, p.Hk / p.kv_rep, D, kDecodeStageKeys))
        return MODA_ERR_CUDA;
    static thread_local int configured_dev = -1;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (configured_dev != dev) {
        if (!set_smem_limit(decode_split_tma_kernel<D, G>, L::kDynamic)) return MODA_ERR_CUDA;
        configured_dev = dev;
    }
    // persistent: one CTA per SM (or per work item when there are fewer)
    const long long items = (long long)p.B * p.Hk * p.S;
    const unsigned grid = unsigned(items < p.num_sms ? items : p.num_sms);
    decode_split_tma_kernel<D, G><<<grid, kDecodeTmaThreads, L::kDynamic, stream>>>(mK, mV, p);
    if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    decode_merge_kernel<D><<<dim3(p.H, p.B), kDecodeMergeThreads, 0, stream>>>(p);
    if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    return MODA_OK;
}
template <int D>
int launch_decode(const DecodeParams& p, cudaStream_t stream) {
    switch (p.H / p.Hk) {
        case 1: return launch_decode_g<D, 1>(p, stream);
        case 2: return launch_decode_g<D, 2>(p, stream);
        case 3: return launch_decode_g<D, 3>(p, stream);
        case 4: return launch_decode_g<D, 4>(p, stream);
        case 5: return launch_decode_g<D, 5>(p, stream);
        case 6: return launch_decode_g<D, 6>(p, stream);
        case 7: return launch_decode_g<D, 7>(p, stream);
        case 8: return launch_decode_g<D, 8>(p, stream);
        default: return MODA_ERR_BAD_GROUP;
    }
}

int device_sm_count(int* out) {
    static thread_local int cached_dev = -1, cached_sms = 0;
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (dev != cached_dev) {
        int sms = 0;
        if (!cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return MODA_ERR_CUDA;
        cached_dev = dev; cached_sms = sms;
    }
    *out = cached_sms;
    return MODA_OK;
}

// The decode step behind its three entry points: contiguous cache with one length, contiguous cache with a
// length per sequence, paged cache (T_cap then counts pages).
int decode_common(const void* q, const void* K, const void* V, const int* seq_lens, const int* block_table,
                  const void* depth_kv_token, int B, int T_kv, int T_cap, int page_size, int max_blocks,
                  int H, int H_kv, int d, int l, float scale,
                  void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream) {
    const bool paged = block_table != nullptr;
    if (B < 1 || T_kv < 1 || H < 1 || (!paged && T_cap < T_kv)) return MODA_ERR_BAD_SHAPE;
    if (d != 64 && d != 128) return MODA_ERR_BAD_HEAD_DIM;
    if (int rc = check_scale(scale)) return rc;
    if ((long long)(paged ? page_size : B) * T_cap > 0x7fffffffLL / H) return MODA_ERR_BAD_SHAPE;
    if (int rc = check_groups(H, H_kv)) return rc;
    if ((long long)B * H * kDecodeMaxSplits > 0x7fffffffLL || B > 65535) return MODA_ERR_BAD_SHAPE;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!q || !K || !V || !O || !LSE || (l > 0 && !depth_kv_token)) return MODA_ERR_NULL_POINTER;
    if ((seq_lens && (reinterpret_cast<uintptr_t>(seq_lens) & 3u)) || (block_table && (reinterpret_cast<uintptr_t>(block_table) & 3u)))
        return MODA_ERR_MISALIGNED;
    if (!aligned16(q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) ||
        (l > 0 && !aligned16(depth_kv_token)))
        return MODA_ERR_MISALIGNED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < decode_workspace_bytes(B, H, d)) return MODA_ERR_WORKSPACE;
    if (int rc = check_device()) return rc;
    int sms = 0;
    if (int rc = device_sm_count(&sms)) return rc;
    DecodeParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.K = static_cast<const __nv_bfloat16*>(K);
    p.V = static_cast<const __nv_bfloat16*>(V);
    p.depth = static_cast<const __nv_bfloat16*>(depth_kv_token);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.LSE = LSE;
    p.part = static_cast<float*>(workspace);
    // 16 or 32 query heads per key/value head: groups of 8 heads that read the same K, V head
    const int kv_rep = (H / H_kv > 8) ? (H / H_kv) / 8 : 1;
    p.B = B; p.T_kv = T_kv; p.T_cap = T_cap; p.H = H; p.Hk = H_kv * kv_rep; p.l = l; p.kv_rep = kv_rep;
    p.seq_lens = seq_lens; p.block_table = block_table; p.page_size = page_size; p.max_blocks = max_blocks;
    const DecodePlan plan = decode_plan(B, p.Hk, T_kv, sms);
    p.S = plan.S; p.keys_per_split = plan.keys_per_split; p.num_sms = sms;
    p.scale_log2 = scale * kDecodeLog2e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_decode<128>(p, st) : launch_decode<64>(p, st);
}

}  // namespace

namespace {
int kv_project_common(const void* X, const void* Wk, const void* Wv, int B, int T, int D_model, int H_kv, int d,
                      void* K_out, void* V_out, void* cache, int slot, void* stream, bool e4m3) {
    if (int rc = check_shape(B, T, H_kv, d)) return rc;
    if (D_model < 64 || D_model % 64 != 0 || (long long)B * T > 0x7fffffffLL / D_model) return MODA_ERR_BAD_SHAPE;
    if (cache != nullptr && (slot < 0 || slot >= MODA_MAX_DEPTH)) return MODA_ERR_BAD_SLOT;
    if (!X || !Wk || !Wv || (K_out == nullptr) != (V_out == nullptr) || (!K_out && !cache)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(X) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(K_out) || !aligned16(V_out) || !aligned16(cache))
        return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* slot_base = nullptr;
    if (cache)
        slot_base = e4m3 ? static_cast<void*>(static_cast<uint8_t*>(cache) + size_t(slot) * cache8_slot_bytes(B, T, H_kv, d))
                         : static_cast<void*>(static_cast<__nv_bfloat16*>(cache) + size_t(slot) * cache_slot_elems(B, T, H_kv, d));
    // d = 64: two heads per CTA (one tensor-core instruction of 256 columns) when the heads pair up
    if (e4m3) {
        if (d == 128) return launch_kv_project<128, 1, true>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st);
        return H_kv % 2 == 0 ? launch_kv_project<64, 2, true>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st)
                             : launch_kv_project<64, 1, true>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st);
    }
    if (d == 128) return launch_kv_project<128, 1>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st);
    return H_kv % 2 == 0 ? launch_kv_project<64, 2>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st)
                         : launch_kv_project<64, 1>(X, Wk, Wv, B, T, D_model, H_kv, K_out, V_out, slot_base, st);
}
}  // namespace

extern "C" {

int moda_version(void) { return 100; }

const char* moda_strerror(int code) {
    switch (code) {
        case MODA_OK: return "ok";
        case MODA_ERR_NULL_POINTER: return "a required pointer is null";
        case MODA_ERR_MISALIGNED: return "a tensor pointer is not 16-byte aligned";
        case MODA_ERR_BAD_SHAPE: return "B, T and H must be >= 1 and the tensor must fit 31-bit row counts";
        case MODA_ERR_BAD_HEAD_DIM: return "head width d must be 64 or 128";
        case MODA_ERR_BAD_DEPTH: return "depth l must be in [0, 256]";
        case MODA_ERR_BAD_SLOT: return "depth slot must be in [0, 256)";
        case MODA_ERR_WORKSPACE: return "workspace is null or too small";
        case MODA_ERR_DEVICE: return "the current CUDA device is not an sm_100 part";
        case MODA_ERR_CUDA: return "a CUDA call failed (see moda_last_cuda_error)";
        case MODA_ERR_DEVICE_TIMEOUT: return "a kernel gave up a bounded wait (see moda_last_status)";
        case MODA_ERR_BAD_GROUP: return "H_kv must divide H with 1 to 8, 16 or 32 query heads per key/value head";
        case MODA_ERR_BAD_SCALE: return "the softmax scale must be finite and at least 1e-20";
        case MODA_ERR_SCRATCH_LIMIT: return "B*H*T exceeds the built-in scratch of moda_attn_bwd_static_scratch (2^20 rows)";
        default: return "unknown error code";
    }
}

int moda_last_cuda_error(void) { return tl_last_cuda_error; }


int moda_selftest_wait_timeout(void* stream) {
    if (int rc = check_device()) return rc;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(1000000ull);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}

int moda_last_status(int clear) {
    int st = 0;
    if (!cuda_ok(cudaDeviceSynchronize())) return MODA_ERR_CUDA;
    if (!cuda_ok(cudaMemcpyFromSymbol(&st, g_moda_status, sizeof(int)))) return MODA_ERR_CUDA;
    if (clear && st != 0) {
        const int zero = 0;
        if (!cuda_ok(cudaMemcpyToSymbol(g_moda_status, &zero, sizeof(int)))) return MODA_ERR_CUDA;
        int dev = 0;
        if (cuda_ok(cudaGetDevice(&dev)) && dev >= 0 && dev < kMaxDevices && g_status_mirror[dev] != nullptr)
            *g_status_mirror[dev] = 0;
    }
    return st;
}

size_t moda_depth_cache_bytes(int B, int T, int H, int d, int l_max) {
    if (check_shape(B, T, H, d) != MODA_OK || l_max < 0 || l_max > MODA_MAX_DEPTH) return 0;
    return size_t(l_max) * cache_slot_elems(B, T, H, d) * 2;
}

int moda_depth_cache_append(void* cache, int B, int T, int H, int d, int slot,
                            const void* K_i, const void* V_i, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (slot < 0 || slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!cache || !K_i || !V_i) return MODA_ERR_NULL_POINTER;
    if (!aligned16(cache) || !aligned16(K_i) || !aligned16(V_i)) return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_cache_copy<128, true>(cache, B, T, H, slot, const_cast<void*>(K_i), const_cast<void*>(V_i), st)
                    : launch_cache_copy<64, true>(cache, B, T, H, slot, const_cast<void*>(K_i), const_cast<void*>(V_i), st);
}

int moda_depth_cache_unpack(const void* cache, int B, int T, int H, int d, int slot,
                            void* K_i, void* V_i, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (slot < 0 || slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!cache || (!K_i && !V_i)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(cache) || !aligned16(K_i) || !aligned16(V_i)) return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_cache_copy<128, false>(const_cast<void*>(cache), B, T, H, slot, K_i, V_i, st)
                    : launch_cache_copy<64, false>(const_cast<void*>(cache), B, T, H, slot, K_i, V_i, st);
}

int moda_attn_fwd(const void* Q, const void* K, const void* V, const void* depth_kv,
                  int B, int T, int H, int d, int l, float scale,
                  void* O, float* LSE, void* stream) {
    return moda_attn_fwd_gqa(Q, K, V, depth_kv, B, T, H, H, d, l, scale, O, LSE, stream);
}

int moda_attn_fwd_gqa(const void* Q, const void* K, const void* V, const void* depth_kv,
                      int B, int T, int H, int H_kv, int d, int l, float scale,
                      void* O, float* LSE, void* stream) {
    return moda_attn_fwd_prefill(Q, K, V, depth_kv, B, T, T, H, H_kv, d, l, scale, O, LSE, stream);
}

int moda_attn_fwd_prefill(const void* Q, const void* K, const void* V, const void* depth_kv,
                          int B, int T_q, int T_kv, int H, int H_kv, int d, int l, float scale,
                          void* O, float* LSE, void* stream) {
    if (int rc = check_shape(B, T_q, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (T_kv < T_q) return MODA_ERR_BAD_SHAPE;
    if (int rc = check_shape(B, T_kv, H, d)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !LSE || (l > 0 && !depth_kv)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) ||
        (l > 0 && !aligned16(depth_kv)))
        return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_fwd<128>(Q, K, V, depth_kv, B, T_q, T_kv, H, H_kv, l, scale, O, LSE, nullptr, st)
                    : launch_fwd<64>(Q, K, V, depth_kv, B, T_q, T_kv, H, H_kv, l, scale, O, LSE, nullptr, st);
}

int moda_attn_fwd_append(const void* Q, const void* K, const void* V, const void* depth_kv,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* O, float* LSE, void* append_cache, int append_slot, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (append_slot < 0 || append_slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!Q || !K || !V || !O || !LSE || !append_cache || (l > 0 && !depth_kv)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) || !aligned16(append_cache) ||
        (l > 0 && !aligned16(depth_kv)))
        return MODA_ERR_MISALIGNED;
    // The slot being written may be one of the slots being read only with one key/value head per query head: a CTA then
    // reads and writes the blocks of its own (b, h, tile) alone, and it writes after its depth warps have finished reading
    // (a fixed-size slot buffer whose oldest or least useful slot is replaced in place).  With grouped heads the other
    // heads of the group read the block that the first head writes.
    if (l > 0 && append_cache == depth_kv && append_slot < l && H_kv != H) return MODA_ERR_BAD_SLOT;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* slot = static_cast<__nv_bfloat16*>(append_cache) + size_t(append_slot) * cache_slot_elems(B, T, H_kv, d);
    return d == 128 ? launch_fwd<128>(Q, K, V, depth_kv, B, T, T, H, H_kv, l, scale, O, LSE, slot, st)
                    : launch_fwd<64>(Q, K, V, depth_kv, B, T, T, H, H_kv, l, scale, O, LSE, slot, st);
}

size_t moda_bwd_workspace_bytes(int B, int T, int H, int d, int l) {
    return moda_bwd_workspace_bytes_gqa(B, T, H, H, d, l);
}

// Enough for either form of the backward (the reproducible split form needs far less than the fused one).
size_t moda_bwd_workspace_bytes_gqa(int B, int T, int H, int H_kv, int d, int l) {
    if (check_shape(B, T, H, d) != MODA_OK || check_groups(H, H_kv) != MODA_OK || l < 0 || l > MODA_MAX_DEPTH) return 0;
    const size_t split = bwd_workspace_bytes_gqa(B, T, H, H_kv, l);
    const size_t fused = bwd_fused_workspace_bytes(B, T, H, d);   // also what the e4m3 and position-major calls take
    return split > fused ? split : fused;
}

int moda_attn_bwd(const void* Q, const void* K, const void* V, const void* depth_kv,
                  const void* O, const void* dO, const float* LSE,
                  int B, int T, int H, int d, int l, float scale,
                  void* dQ, void* dK, void* dV, void* d_depth_kv,
                  void* workspace, size_t workspace_bytes, void* stream) {
    return moda_attn_bwd_stages(Q, K, V, depth_kv, O, dO, LSE, B, T, H, d, l, scale, dQ, dK, dV, d_depth_kv,
                                workspace, workspace_bytes, MODA_BWD_ALL_STAGES, stream);
}

int moda_attn_bwd_stages(const void* Q, const void* K, const void* V, const void* depth_kv,
                         const void* O, const void* dO, const float* LSE,
                         int B, int T, int H, int d, int l, float scale,
                         void* dQ, void* dK, void* dV, void* d_depth_kv,
                         void* workspace, size_t workspace_bytes, int stages, void* stream) {
    return moda_attn_bwd_gqa_stages(Q, K, V, depth_kv, O, dO, LSE, B, T, H, H, d, l, scale, dQ, dK, dV, d_depth_kv,
                                    workspace, workspace_bytes, stages, stream);
}

int moda_attn_bwd_gqa(const void* Q, const void* K, const void* V, const void* depth_kv,
                      const void* O, const void* dO, const float* LSE,
                      int B, int T, int H, int H_kv, int d, int l, float scale,
                      void* dQ, void* dK, void* dV, void* d_depth_kv,
                      void* workspace, size_t workspace_bytes, void* stream) {
    return moda_attn_bwd_gqa_stages(Q, K, V, depth_kv, O, dO, LSE, B, T, H, H_kv, d, l, scale, dQ, dK, dV, d_depth_kv,
                                    workspace, workspace_bytes, MODA_BWD_ALL_STAGES, stream);
}

int moda_attn_bwd_gqa_stages(const void* Q, const void* K, const void* V, const void* depth_kv,
                             const void* O, const void* dO, const float* LSE,
                             int B, int T, int H, int H_kv, int d, int l, float scale,
                             void* dQ, void* dK, void* dV, void* d_depth_kv,
                             void* workspace, size_t workspace_bytes, int stages, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if ((stages & MODA_BWD_ALL_STAGES) == 0 || stages < 0 ||
        stages > (MODA_BWD_ALL_STAGES | MODA_BWD_ACCUMULATE_DEPTH | MODA_BWD_DETERMINISTIC))
        return MODA_ERR_BAD_SHAPE;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV || (l > 0 && (!depth_kv || !d_depth_kv)))
        return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(LSE) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) ||
        (l > 0 && (!aligned16(depth_kv) || !aligned16(d_depth_kv))))
        return MODA_ERR_MISALIGNED;
    const bool deterministic = (stages & MODA_BWD_DETERMINISTIC) != 0;
    const size_t need = bwd_uses_fused(d, H / H_kv, l, deterministic) ? bwd_fused_workspace_bytes(B, T, H, d)
                                                                       : bwd_workspace_bytes_gqa(B, T, H, H_kv, l);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return MODA_ERR_WORKSPACE;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    BwdArgs a;
    a.deterministic = deterministic;
    a.Q = Q; a.K = K; a.V = V; a.depth_kv = depth_kv; a.O = O; a.dO = dO; a.LSE = LSE;
    a.B = B; a.T = T; a.H = H; a.Hk = H_kv; a.l = l; a.scale = scale;
    a.dQ = dQ; a.dK = dK; a.dV = dV; a.d_depth_kv = d_depth_kv; a.workspace = workspace;
    a.accumulate_depth = (stages & MODA_BWD_ACCUMULATE_DEPTH) != 0;
    return d == 128 ? launch_bwd<128>(a, stages, st) : launch_bwd<64>(a, stages, st);
}

// ---- depth cache in e4m3 with a scale per row ----
size_t moda_depth_cache_e4m3_bytes(int B, int T, int H, int d, int l_max) {
    if (check_shape(B, T, H, d) != MODA_OK || l_max < 0 || l_max > MODA_MAX_DEPTH) return 0;
    return size_t(l_max) * cache8_slot_bytes(B, T, H, d);
}

int moda_depth_cache_append_e4m3(void* cache, int B, int T, int H, int d, int slot,
                                 const void* K_i, const void* V_i, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (slot < 0 || slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!cache || !K_i || !V_i) return MODA_ERR_NULL_POINTER;
    if (!aligned16(cache) || !aligned16(K_i) || !aligned16(V_i)) return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* base = static_cast<uint8_t*>(cache) + size_t(slot) * cache8_slot_bytes(B, T, H, d);
    const unsigned grid = unsigned(B) * H * num_tiles(T) * 2;
    if (d == 128)
        depth_cache_quant_kernel<128><<<grid, 256, 0, st>>>(base, static_cast<const uint4*>(K_i), static_cast<const uint4*>(V_i), T, H);
    else
        depth_cache_quant_kernel<64><<<grid, 256, 0, st>>>(base, static_cast<const uint4*>(K_i), static_cast<const uint4*>(V_i), T, H);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}

int moda_attn_fwd_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                       int B, int T, int H, int H_kv, int d, int l, float scale,
                       void* O, float* LSE, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !LSE || (l > 0 && !depth_kv_e4m3)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) ||
        (l > 0 && !aligned16(depth_kv_e4m3)))
        return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_fwd<128>(Q, K, V, depth_kv_e4m3, B, T, T, H, H_kv, l, scale, O, LSE, nullptr, st, kCacheE4m3)
                    : launch_fwd<64>(Q, K, V, depth_kv_e4m3, B, T, T, H, H_kv, l, scale, O, LSE, nullptr, st, kCacheE4m3);
}

int moda_attn_fwd_append_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                              int B, int T, int H, int H_kv, int d, int l, float scale,
                              void* O, float* LSE, void* append_cache_e4m3, int append_slot, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (append_slot < 0 || append_slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!Q || !K || !V || !O || !LSE || !append_cache_e4m3 || (l > 0 && !depth_kv_e4m3)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) || !aligned16(append_cache_e4m3) ||
        (l > 0 && !aligned16(depth_kv_e4m3)))
        return MODA_ERR_MISALIGNED;
    // as in moda_attn_fwd_append: a slot that the call also reads may be written only with one key/value head per query head
    if (l > 0 && append_cache_e4m3 == depth_kv_e4m3 && append_slot < l && H_kv != H) return MODA_ERR_BAD_SLOT;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* slot = static_cast<uint8_t*>(append_cache_e4m3) + size_t(append_slot) * cache8_slot_bytes(B, T, H_kv, d);
    // Quantising a row costs the depth warps about as many instructions as eight depth slots do.  On long sequences that
    // disappears under the key loop (64K: + 0.07 ms against 0.19 ms for a separate pass); on short ones the depth warps
    // set the pace and the separate HBM-bound pass is cheaper (8K, l = 16: 0.06 ms against + 0.14 ms), so the quantiser
    // then runs as its own launch behind the forward (same bytes; still after every read of the cache by this call).
    const bool fused = T >= 32768;
    const int rc = d == 128 ? launch_fwd<128>(Q, K, V, depth_kv_e4m3, B, T, T, H, H_kv, l, scale, O, LSE, fused ? slot : nullptr, st, kCacheE4m3)
                            : launch_fwd<64>(Q, K, V, depth_kv_e4m3, B, T, T, H, H_kv, l, scale, O, LSE, fused ? slot : nullptr, st, kCacheE4m3);
    if (rc != MODA_OK || fused) return rc;
    return moda_depth_cache_append_e4m3(append_cache_e4m3, B, T, H_kv, d, append_slot, K, V, stream);
}

int moda_attn_bwd_e4m3(const void* Q, const void* K, const void* V, const void* depth_kv_e4m3,
                       const void* O, const void* dO, const float* LSE,
                       int B, int T, int H, int d, int l, float scale,
                       void* dQ, void* dK, void* dV, void* d_depth_kv,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV || (l > 0 && (!depth_kv_e4m3 || !d_depth_kv)))
        return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(LSE) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) ||
        (l > 0 && (!aligned16(depth_kv_e4m3) || !aligned16(d_depth_kv))))
        return MODA_ERR_MISALIGNED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < bwd_fused_workspace_bytes(B, T, H, d)) return MODA_ERR_WORKSPACE;
    if (int rc = check_device()) return rc;
    BwdArgs a;
    a.fp8_cache = true;
    a.Q = Q; a.K = K; a.V = V; a.depth_kv = depth_kv_e4m3; a.O = O; a.dO = dO; a.LSE = LSE;
    a.B = B; a.T = T; a.H = H; a.Hk = H; a.l = l; a.scale = scale;
    a.dQ = dQ; a.dK = dK; a.dV = dV; a.d_depth_kv = d_depth_kv; a.workspace = workspace;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_bwd_fused<128>(a, MODA_BWD_ALL_STAGES, st) : launch_bwd_fused<64>(a, MODA_BWD_ALL_STAGES, st);
}

// ---- position-major depth cache for grouped-query calls ----
int moda_depth_cache_append_pm(void* cache, int B, int T, int H, int d, int slot,
                               const void* K_i, const void* V_i, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (slot < 0 || slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!cache || !K_i || !V_i) return MODA_ERR_NULL_POINTER;
    if (!aligned16(cache) || !aligned16(K_i) || !aligned16(V_i)) return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_cache_pm_copy<128, true>(cache, B, T, H, slot, const_cast<void*>(K_i), const_cast<void*>(V_i), st)
                    : launch_cache_pm_copy<64, true>(cache, B, T, H, slot, const_cast<void*>(K_i), const_cast<void*>(V_i), st);
}

int moda_depth_cache_unpack_pm(const void* cache, int B, int T, int H, int d, int slot,
                               void* K_i, void* V_i, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (slot < 0 || slot >= MODA_MAX_DEPTH) return MODA_ERR_BAD_SLOT;
    if (!cache || (!K_i && !V_i)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(cache) || !aligned16(K_i) || !aligned16(V_i)) return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_cache_pm_copy<128, false>(const_cast<void*>(cache), B, T, H, slot, K_i, V_i, st)
                    : launch_cache_pm_copy<64, false>(const_cast<void*>(cache), B, T, H, slot, K_i, V_i, st);
}

int moda_attn_fwd_gqa_pm(const void* Q, const void* K, const void* V, const void* depth_kv_pm,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* O, float* LSE, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (H == H_kv) return MODA_ERR_BAD_GROUP;                 // the per-position kernels need at least two heads per group
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !LSE || (l > 0 && !depth_kv_pm)) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE) ||
        (l > 0 && !aligned16(depth_kv_pm)))
        return MODA_ERR_MISALIGNED;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_fwd<128>(Q, K, V, depth_kv_pm, B, T, T, H, H_kv, l, scale, O, LSE, nullptr, st, kCachePm)
                    : launch_fwd<64>(Q, K, V, depth_kv_pm, B, T, T, H, H_kv, l, scale, O, LSE, nullptr, st, kCachePm);
}

int moda_attn_bwd_gqa_pm(const void* Q, const void* K, const void* V, const void* depth_kv_pm,
                         const void* O, const void* dO, const float* LSE,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         void* dQ, void* dK, void* dV, void* d_depth_kv_pm,
                         void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (int rc = check_groups(H, H_kv)) return rc;
    if (H == H_kv) return MODA_ERR_BAD_GROUP;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV || (l > 0 && (!depth_kv_pm || !d_depth_kv_pm)))
        return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(LSE) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) ||
        (l > 0 && (!aligned16(depth_kv_pm) || !aligned16(d_depth_kv_pm))))
        return MODA_ERR_MISALIGNED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < bwd_fused_workspace_bytes(B, T, H, d)) return MODA_ERR_WORKSPACE;
    if (int rc = check_device()) return rc;
    BwdArgs a;
    a.pm_cache = true;
    a.Q = Q; a.K = K; a.V = V; a.depth_kv = depth_kv_pm; a.O = O; a.dO = dO; a.LSE = LSE;
    a.B = B; a.T = T; a.H = H; a.Hk = H_kv; a.l = l; a.scale = scale;
    a.dQ = dQ; a.dK = dK; a.dV = dV; a.d_depth_kv = d_depth_kv_pm; a.workspace = workspace;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_bwd_fused<128>(a, MODA_BWD_ALL_STAGES, st) : launch_bwd_fused<64>(a, MODA_BWD_ALL_STAGES, st);
}

int moda_kv_project_append(const void* X, const void* Wk, const void* Wv,
                           int B, int T, int D_model, int H_kv, int d,
                           void* K_out, void* V_out, void* cache, int slot, void* stream) {
    return kv_project_common(X, Wk, Wv, B, T, D_model, H_kv, d, K_out, V_out, cache, slot, stream, false);
}

int moda_kv_project_append_e4m3(const void* X, const void* Wk, const void* Wv,
                                int B, int T, int D_model, int H_kv, int d,
                                void* K_out, void* V_out, void* cache_e4m3, int slot, void* stream) {
    return kv_project_common(X, Wk, Wv, B, T, D_model, H_kv, d, K_out, V_out, cache_e4m3, slot, stream, true);
}

size_t moda_depth_slot_mass_workspace_bytes(int B, int T, int H, int l) {
    if (B < 1 || T < 1 || H < 1 || l < 0 || l > MODA_MAX_DEPTH) return 0;
    return size_t(B) * H * num_tiles(T) * size_t(l > 0 ? l : 1) * sizeof(float);
}

int moda_depth_slot_mass(const void* Q, const void* depth_kv, const float* LSE,
                         int B, int T, int H, int H_kv, int d, int l, float scale,
                         float* mass, void* workspace, size_t workspace_bytes, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (H_kv < 1 || H % H_kv != 0) return MODA_ERR_BAD_GROUP;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if (l == 0) return MODA_OK;                    // no slots: nothing to write
    if (!Q || !depth_kv || !LSE || !mass) return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(depth_kv) || !aligned16(LSE) || !aligned16(mass)) return MODA_ERR_MISALIGNED;
    if (!workspace || !aligned16(workspace) || workspace_bytes < moda_depth_slot_mass_workspace_bytes(B, T, H, l))
        return MODA_ERR_WORKSPACE;
    if (int rc = check_device()) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MassParams p;
    p.Q = static_cast<const __nv_bfloat16*>(Q);
    p.depth_kv = static_cast<const __nv_bfloat16*>(depth_kv);
    p.LSE = LSE;
    p.partial = static_cast<float*>(workspace);
    p.mass = mass;
    p.B = B; p.T = T; p.H = H; p.G = H / H_kv; p.l = l;
    p.scale_log2 = scale * kLog2e;
    const unsigned grid = unsigned(B) * H * num_tiles(T);
    if (d == 128) depth_slot_mass_kernel<128><<<grid, kTileRows * 4, 0, st>>>(p);
    else depth_slot_mass_kernel<64><<<grid, kTileRows * 2, 0, st>>>(p);
    if (!cuda_ok(cudaGetLastError())) return MODA_ERR_CUDA;
    const long long n = (long long)B * H * l;
    depth_slot_mass_reduce_kernel<<<unsigned((n + 255) / 256), 256, 0, st>>>(p);
    return cuda_ok(cudaGetLastError()) ? MODA_OK : MODA_ERR_CUDA;
}

size_t moda_decode_workspace_bytes(int B, int H, int d) {
    if (B < 1 || H < 1 || (d != 64 && d != 128)) return 0;
    return decode_workspace_bytes(B, H, d);
}

int moda_attn_decode(const void* q, const void* K, const void* V, const void* depth_kv_token,
                     int B, int T_kv, int T_cap, int H, int H_kv, int d, int l, float scale,
                     void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream) {
    return decode_common(q, K, V, nullptr, nullptr, depth_kv_token, B, T_kv, T_cap, 0, 0, H, H_kv, d, l, scale,
                         O, LSE, workspace, workspace_bytes, stream);
}

int moda_attn_decode_varlen(const void* q, const void* K, const void* V, const int* seq_lens,
                            const void* depth_kv_token,
                            int B, int max_seq_len, int T_cap, int H, int H_kv, int d, int l, float scale,
                            void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream) {
    if (!seq_lens) return MODA_ERR_NULL_POINTER;
    return decode_common(q, K, V, seq_lens, nullptr, depth_kv_token, B, max_seq_len, T_cap, 0, 0, H, H_kv, d, l, scale,
                         O, LSE, workspace, workspace_bytes, stream);
}

int moda_attn_decode_paged(const void* q, const void* K_pages, const void* V_pages,
                           const int* block_table, const int* seq_lens, const void* depth_kv_token,
                           int B, int max_seq_len, int page_size, int num_pages, int max_blocks_per_seq,
                           int H, int H_kv, int d, int l, float scale,
                           void* O, float* LSE, void* workspace, size_t workspace_bytes, void* stream) {
    if (!block_table || !seq_lens) return MODA_ERR_NULL_POINTER;
    if (page_size < kDecodeStageKeys || page_size % kDecodeStageKeys != 0 || num_pages < 1 || max_blocks_per_seq < 1 ||
        (long long)max_blocks_per_seq * page_size < max_seq_len)
        return MODA_ERR_BAD_SHAPE;
    return decode_common(q, K_pages, V_pages, seq_lens, block_table, depth_kv_token, B, max_seq_len, num_pages, page_size,
                         max_blocks_per_seq, H, H_kv, d, l, scale, O, LSE, workspace, workspace_bytes, stream);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Backward without a caller workspace: the row terms live in an array inside the library image.
// ------------------------------------------------------------------------------------------
namespace {

// In host code this name is only a handle for the runtime, not a device address: the address
// each GPU gave the array is looked up once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_rowterms[MODA_STATIC_SCRATCH_ROWS];

std::mutex g_static_mutex;
float* g_static_rowterms_addr[kMaxDevices] = {};

// Device address of the built-in scratch on the current device (looked up on first use).
int static_scratch_for_current_device(float** out) {
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return MODA_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MODA_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_rowterms_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (!cuda_ok(cudaGetSymbolAddress(&ptr, g_static_rowterms)) || ptr == nullptr) return MODA_ERR_CUDA;
        g_static_rowterms_addr[dev] = static_cast<float*>(ptr);
    }
    *out = g_static_rowterms_addr[dev];
    return MODA_OK;
}

}  // namespace

extern "C" int moda_attn_bwd_static_scratch(const void* Q, const void* K, const void* V, const void* depth_kv,
                                            const void* O, const void* dO, const float* LSE,
                                            int B, int T, int H, int d, int l, float scale,
                                            void* dQ, void* dK, void* dV, void* d_depth_kv, void* stream) {
    if (int rc = check_shape(B, T, H, d)) return rc;
    if (int rc = check_scale(scale)) return rc;
    if (l < 0 || l > MODA_MAX_DEPTH) return MODA_ERR_BAD_DEPTH;
    if ((long long)B * H * T > (long long)MODA_STATIC_SCRATCH_ROWS) return MODA_ERR_SCRATCH_LIMIT;
    if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV || (l > 0 && (!depth_kv || !d_depth_kv)))
        return MODA_ERR_NULL_POINTER;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) || !aligned16(LSE) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) ||
        (l > 0 && (!aligned16(depth_kv) || !aligned16(d_depth_kv))))
        return MODA_ERR_MISALIGNED;
    if (int rc = check_device(/*may_allocate=*/false)) return rc;
    float* scratch = nullptr;
    if (int rc = static_scratch_for_current_device(&scratch)) return rc;
    BwdArgs a;
    a.Q = Q; a.K = K; a.V = V; a.depth_kv = depth_kv; a.O = O; a.dO = dO; a.LSE = LSE;
    a.B = B; a.T = T; a.H = H; a.Hk = H; a.l = l; a.scale = scale;
    a.dQ = dQ; a.dK = dK; a.dV = dV; a.d_depth_kv = d_depth_kv; a.workspace = scratch;
    a.deterministic = true;                  // the split form: its only scratch is the row terms, which fit the built-in array
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 128 ? launch_bwd<128>(a, MODA_BWD_ALL_STAGES, st) : launch_bwd<64>(a, MODA_BWD_ALL_STAGES, st);
}
