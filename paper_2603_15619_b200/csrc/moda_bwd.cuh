// MoDA backward kernels for sm_100a.  The paper prints no backward pass; these kernels
// evaluate the derivative of the Sec. 2.2 operator.  With P = exp(S - LSE) (sequence),
// R = exp(U - LSE) (depth), D_t = <dO_t, O_t>:
//
//   dS = P o (dO V^T - D),   dU_i = R_i (<dO, Vd_i> - D)
//   dQ = scale (dS K + sum_i dU_i Kd_i)     dK = scale dS^T Q     dV = P^T dO
//   dKd_i = scale dU_i Q                    dVd_i = R_i dO        (row-local)
//
// Three launches on the caller's stream, all deterministic (no atomics):
//   1. bwd_delta_kernel      D_t for every row (fp32 workspace).
//   2. moda_bwd_dq_kernel    one CTA per 128-query tile, loops over 64-key tiles: S and
//                            dP = dO V^T on tcgen05, dS written back to TMEM as bf16, dQ += dS K
//                            accumulated in TMEM.  A second warpgroup does the whole depth
//                            backward for the tile's rows on the CUDA cores (reads the depth
//                            cache, writes dKd / dVd in cache layout) and parks its dQ share in
//                            TMEM; the epilogue adds the two.
//   3. moda_bwd_dkdv_kernel  one CTA per 128-key tile, loops over 64-query tiles in the
//                            transposed formulation (S^T = K Q^T, dP^T = V dO^T) so that
//                            P^T and dS^T are TMEM A-operands of dV += P^T dO, dK += dS^T Q.
//
// Grouped-query attention (H query heads on H / G key/value heads): dK, dV sum over the G heads
// inside the dK/dV kernel (its loop runs over the group's (head, query tile) pairs); the depth
// gradients sum over heads that live in different CTAs of the dQ kernel, so that kernel then only
// leaves its per-row factors and depth_grad_group_kernel (a fourth launch) forms the sums.
#pragma once

#include "moda_cache.cuh"
#include "moda_fwd.cuh"
#include "sm100_ptx.cuh"

namespace moda {

struct BwdArgs {
    const void *Q, *K, *V, *depth_kv, *O, *dO;
    const float* LSE;
    int B, T, H, Hk, l;          // H query heads on Hk key/value heads
    float scale;
    void *dQ, *dK, *dV, *d_depth_kv, *workspace;
    bool accumulate_depth = false;   // add the depth gradients to d_depth_kv instead of overwriting it
    bool deterministic = false;      // split form (bit-reproducible) instead of the fused form
    bool pm_cache = false;           // depth_kv and d_depth_kv are position-major (grouped-query calls, fused form, per-position depth kernel)
    bool fp8_cache = false;          // depth_kv holds e4m3 codes + row scales (fused form, one KV head per query head only)
};

inline size_t bwd_workspace_bytes(int B, int T, int H) {
    return (size_t(B) * H * T * 4 + 15) & ~size_t(15);
}
// Grouped-query backward: the row terms D_t, then R_i and dU_i of every (row, slot, head).
inline size_t bwd_workspace_bytes_gqa(int B, int T, int H, int Hk, int l) {
    const size_t base = bwd_workspace_bytes(B, T, H);
    if (H == Hk) return base;
    return base + size_t(B) * Hk * num_tiles(T) * l * 2 * kTileRows * (H / Hk) * 4;
}

__device__ __forceinline__ float dot8_bf16(const uint4& a, const uint4& b) {
    float acc = bf16_lo_to_f32(a.x) * bf16_lo_to_f32(b.x);
    acc = fmaf(bf16_hi_to_f32(a.x), bf16_hi_to_f32(b.x), acc);
    acc = fmaf(bf16_lo_to_f32(a.y), bf16_lo_to_f32(b.y), acc);
    acc = fmaf(bf16_hi_to_f32(a.y), bf16_hi_to_f32(b.y), acc);
    acc = fmaf(bf16_lo_to_f32(a.z), bf16_lo_to_f32(b.z), acc);
    acc = fmaf(bf16_hi_to_f32(a.z), bf16_hi_to_f32(b.z), acc);
    acc = fmaf(bf16_lo_to_f32(a.w), bf16_lo_to_f32(b.w), acc);
    acc = fmaf(bf16_hi_to_f32(a.w), bf16_hi_to_f32(b.w), acc);
    return acc;
}

// D_t = <dO_t, O_t>, one group of d/8 lanes per row of the [B][T][H] row space; written as [B][H][T].
template <int D>
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const uint4* __restrict__ O, const uint4* __restrict__ dO, float* __restrict__ delta,
                 int B, int T, int H) {
    constexpr int CH = D / 8;
    constexpr int ROWS = 256 / CH;
    const long long nrows = (long long)B * T * H;
    const long long row = (long long)blockIdx.x * ROWS + threadIdx.x / CH;
    const int c = threadIdx.x % CH;
    float acc = 0.f;
    if (row < nrows) acc = dot8_bf16(O[row * CH + c], dO[row * CH + c]);
#pragma unroll
    for (int off = CH / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (row < nrows && c == 0) {
        const int h = int(row % H);
        const long long bt = row / H;
        const int t = int(bt % T);
        const int b = int(bt / T);
        delta[(size_t(b) * H + h) * T + t] = acc;
    }
}

// =====================================================================================
// dQ + depth gradients
// =====================================================================================
// 640 threads: warps 0-3 and 4-7 form dS (each warpgroup takes 32 of a tile's 64 key columns) and
// run the epilogue, warps 8-11 do the depth backward, warp 12 is the TMA producer, warp 13 the
// depth-cache producer, and the three contractions of a tile are issued by three threads on three
// schedulers (warp 16: S = Q K^T, warp 17: dP = dO V^T, warp 18: dQ += dS K), ordered by mbarriers only.
constexpr int kBwdDqThreads = 640;
constexpr int kKeyTile = 64;     // keys per inner tile of the dQ kernel / queries per inner tile of the dK,dV kernel

// The depth backward walks the slots in groups of kDepthGroup: keys (scores), values, keys again
// (dQ share, dKd).  The second visit of a group's keys comes a few hundred KiB per SM after the
// first, so it is served by L2 and the depth cache crosses HBM once; the per-slot row terms only
// need kDepthGroup entries of shared memory.
constexpr int kDepthGroup = 4;

// KVS = stages of the [K_j | V_j] ring.  Three keep the tensor pipe fed on long sequences; two leave
// room for a deeper depth ring (more HBM reads in flight per SM), which is what bounds shapes whose
// depth cache outweighs the sequence work (the host picks, see launch_bwd).
template <int D, int KVS>
struct DqSmem {
    static constexpr int kTileBytes = kTileRows * D * 2;             // 128 x D
    static constexpr int kSubBytes = kTileRows * 128;                // 128 x 64 sub-tile
    static constexpr int kHalfTileBytes = kKeyTile * D * 2;          // 64 x D
    static constexpr int kHalfSubBytes = kKeyTile * 128;             // 64 x 64 sub-tile
    static constexpr int kStages = KVS;
    static constexpr int kQ = 0;
    static constexpr int kdO = kQ + kTileBytes;
    static constexpr int kKV = kdO + kTileBytes;                     // stages of [K_j | V_j]
    static constexpr int kU = kKV + kStages * 2 * kHalfTileBytes;    // [kDepthGroup][128] fp32: u_i, then R_i
    static constexpr int kDr = kU + kDepthGroup * kTileRows * 4;     // [kDepthGroup][128] fp32: <dO,Vd_i>, then dU_i
    static constexpr int kRing = kDr + kDepthGroup * kTileRows * 4;  // depth units: 8 chunks x 128 rows x 16 B
    static constexpr int kUnitBytes = 8 * kTileRows * 16;
    static constexpr int kNumBars = 32;
    static constexpr int kSmemLimit = 232448;                        // 227 KiB per CTA on sm_100
    static constexpr int kRingFit = (kSmemLimit - 1024 - kRing - kNumBars * 8 - 16) / kUnitBytes;
    static constexpr int kRingStages = kRingFit < 8 ? kRingFit : 8;  // every unit that fits, at most 8
    static constexpr int kBars = kRing + kRingStages * kUnitBytes;
    static constexpr int kMisc = kBars + kNumBars * 8;
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static_assert(kRingStages >= 3, "depth ring too shallow");
};

enum DqBar : int {
    kDqBarQ = 0,
    kDqBarKVFull = 1,    // +stage (3)
    kDqBarKVEmpty = 4,   // +stage (3): dQ_j complete (K_j, V_j and the score buffer are free)
    kDqBarSFull = 7,     // +buffer (2), count 2: S_j and dP_j complete
    kDqBarPFull = 9,     // +buffer (2), count 256: dS_j written (and dP_j consumed)
    kDqBarFinal = 11,
    kDqBarDepth = 12,
    kDqBarDrain = 13,    // +issuer (3): abort path only
    kDqBarDFull = 16,    // +ring stage (<= 8)
    kDqBarDEmpty = 24,   // +ring stage (<= 8)
};

struct DqParams {
    const __nv_bfloat16* depth_kv;
    __nv_bfloat16* d_depth_kv;
    const float* LSE;
    const float* delta;
    int B, T, H, l;     // H = number of query heads
    int G;              // query heads per key/value head
    int accumulate;     // nonzero: depth gradients are added to d_depth_kv (bf16 adds in L2)
    // G == 1: the depth gradients are written by this kernel (null here).  G > 1: they are sums
    // over the heads of a group, so the kernel only leaves its per-row factors here, R_i and dU_i
    // as [b][hk][tile][slot][{R, dU}][g][row 128] fp32, and depth_grad_group_kernel forms the sums.
    float* depth_rowterms;
    float scale, scale_log2;
};

// bf16x2 product with both factors already packed.
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

template <int D, int KVS>
__global__ void __launch_bounds__(kBwdDqThreads, 1)
moda_bwd_dq_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
                   const __grid_constant__ CUtensorMap mapK64, const __grid_constant__ CUtensorMap mapV64,
                   const __grid_constant__ CUtensorMap mapdQ, const DqParams p) {
    using L = DqSmem<D, KVS>;
    constexpr int NSUB = D / 64;
    constexpr int CH = D / 8;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0, kColdP = 128, kColdQ = 256, kColdQd = 384;

    if (g_moda_status != 0) return;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    float* sU = reinterpret_cast<float*>(smem + L::kU);
    float* sDr = reinterpret_cast<float*>(smem + L::kDr);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar = [&](int i) { return sbase + L::kBars + 8u * uint32_t(i); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nq = num_tiles(p.T);
    const TileCoord tc = tile_coord(blockIdx.x, nq, p.H, p.G);   // the heads of a group are adjacent CTAs
    const int b = tc.b, h = tc.h, hk = tc.hk, qt = tc.qt;
    const int Hk = p.H / p.G;
    const int q0 = qt * kTileRows;
    const int n_kv = min(2 * (qt + 1), (p.T + kKeyTile - 1) / kKeyTile);   // 64-key tiles at or below the diagonal

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(kDqBarQ), 1);
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar(kDqBarKVFull + s), 1);
            mbar_init(bar(kDqBarKVEmpty + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kDqBarSFull + s), 2);
            mbar_init(bar(kDqBarPFull + s), 256);
        }
        mbar_init(bar(kDqBarFinal), 1);
        mbar_init(bar(kDqBarDepth), 128);
        for (int s = 0; s < 3; ++s) mbar_init(bar(kDqBarDrain + s), 1);
        for (int s = 0; s < L::kRingStages; ++s) {
            mbar_init(bar(kDqBarDFull + s), 1);
            mbar_init(bar(kDqBarDEmpty + s), 128);
        }
        fence_mbar_init();
    }
    if (warp == 16) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Abort path of an issuing thread: wait (bounded) until its own MMAs have drained.
    auto drain_on_abort = [&](int which) {
        if (*abort_flag != 0) {
            umma_commit(bar(kDqBarDrain + which));
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(bar(kDqBarDrain + which), 0) && globaltimer_ns() - t0 < 20000000ull) {}
        }
    };

    if (warp < 8) {
        // =========================== P, dS and the dQ epilogue ===========================
        setmaxnreg_inc<104>();
        const int hc = warp >> 2;                    // which 32 key columns of every tile
        const int r = tid & 127;
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        const bool valid = q0 + r < p.T;
        const size_t row_idx = (size_t(b) * p.H + h) * p.T + q0 + r;
        const float neg_lse2 = valid ? -p.LSE[row_idx] * kLog2e : -INFINITY;   // invalid rows get P = 0
        const float delta = valid ? p.delta[row_idx] : 0.f;
        for (int j = 0; j < n_kv; ++j) {
            const int buf = j & 1;
            mbar_wait(bar(kDqBarSFull + buf), (j >> 1) & 1, abort_flag, 50);
            tc_fence_after_sync();
            const int koff = j * kKeyTile + hc * 32 - q0;    // key of column c is visible to row r iff koff + c <= r
            const bool masked = koff + 31 > 0;
            uint32_t sv[32], gv[32];
            tmem_ld32(tmem + lane_addr + kColS + buf * 64 + hc * 32, sv);
            tmem_ld32(tmem + lane_addr + kColdP + buf * 64 + hc * 32, gv);
            tmem_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                float pa = fast_exp2(fmaf(__uint_as_float(sv[2 * i]), p.scale_log2, neg_lse2));
                float pb = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 1]), p.scale_log2, neg_lse2));
                if (masked) {
                    if (koff + 2 * i > r) pa = 0.f;
                    if (koff + 2 * i + 1 > r) pb = 0.f;
                }
                pk[i] = pack_bf16x2(pa * (__uint_as_float(gv[2 * i]) - delta), pb * (__uint_as_float(gv[2 * i + 1]) - delta));
            }
            // dS_j (bf16, two per column) overlays S_j: each warpgroup writes over the first 16 of the
            // 32 columns it has just read itself, so the two never touch each other's scores.
            tmem_st16(tmem + lane_addr + kColS + buf * 64 + hc * 32, pk);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(kDqBarPFull + buf));
        }
        mbar_wait(bar(kDqBarFinal), 0, abort_flag, 51);
        tc_fence_after_sync();
        if (p.l > 0) {
            mbar_wait(bar(kDqBarDepth), 0, abort_flag, 52);
            tc_fence_after_sync();
        }
        // first warpgroup converts the first half of the feature columns, the second the rest
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {
            const int c = hc * (D / 64) + cc;
            uint32_t o[32];
            tmem_ld32(tmem + lane_addr + kColdQ + c * 32, o);
            tmem_wait_ld();
            float of[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) of[i] = __uint_as_float(o[i]);
            if (p.l > 0) {
                uint32_t od[32];
                tmem_ld32(tmem + lane_addr + kColdQd + c * 32, od);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) of[i] += __uint_as_float(od[i]);
            }
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint4 v;
                v.x = pack_bf16x2(of[8 * g + 0] * p.scale, of[8 * g + 1] * p.scale);
                v.y = pack_bf16x2(of[8 * g + 2] * p.scale, of[8 * g + 3] * p.scale);
                v.z = pack_bf16x2(of[8 * g + 4] * p.scale, of[8 * g + 5] * p.scale);
                v.w = pack_bf16x2(of[8 * g + 6] * p.scale, of[8 * g + 7] * p.scale);
                *reinterpret_cast<uint4*>(smem + L::kQ + swz_chunk_offset(r, c * 4 + g)) = v;
            }
        }
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0) {
#pragma unroll
            for (int s = 0; s < NSUB; ++s) tma_store_4d(&mapdQ, sbase + L::kQ + s * L::kSubBytes, s * 64, h, q0, b);
            tma_store_commit();
            tma_store_wait_all();
        }
    } else if (warp < 12) {
        // =========================== depth backward (row-local) ===========================
        setmaxnreg_inc<176>();
        if (p.l > 0) {
            const int r = tid - 256;
            const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
            const bool valid = q0 + r < p.T;
            const size_t row_idx = (size_t(b) * p.H + h) * p.T + q0 + r;
            const float neg_lse2 = valid ? -p.LSE[row_idx] * kLog2e : -INFINITY;
            const float delta = valid ? p.delta[row_idx] : 0.f;
            const size_t slot_stride = cache_slot_elems(p.B, p.T, Hk, D) / 8;           // in uint4
            const size_t blk = (((size_t(b) * Hk + hk) * nq + qt) * 2) * (kTileRows * CH) + r;
            // Grouped-query launches leave R_i and dU_i of this row for depth_grad_group_kernel
            // instead of writing depth gradients (which are sums over the heads of the group).
            const bool store_grads = p.depth_rowterms == nullptr;
            const bool accumulate = p.accumulate != 0;
            float* rt_row = store_grads ? nullptr
                : p.depth_rowterms + (((size_t(b) * Hk + hk) * nq + qt) * p.l * 2) * (kTileRows * p.G) + (h - hk * p.G) * kTileRows + r;
            uint4* gK = reinterpret_cast<uint4*>(p.d_depth_kv) + blk;
            uint4* gV = gK + kTileRows * CH;
            mbar_wait(bar(kDqBarQ), 0, abort_flag, 60);

            int unit = 0;                                 // running index into the producer's unit sequence
            // Reads this thread's 8 x 16 bytes of the next depth unit from the ring and frees the stage.
            auto take_unit = [&](uint4 (&dst)[8]) {
                const int st = unit % L::kRingStages;
                mbar_wait(bar(kDqBarDFull + st), (unit / L::kRingStages) & 1, abort_flag, 61);
                const uint8_t* src = smem + L::kRing + st * L::kUnitBytes + r * 16;
#pragma unroll
                for (int c = 0; c < 8; ++c) dst[c] = *reinterpret_cast<const uint4*>(src + c * (kTileRows * 16));
                // The stage is refilled by the async proxy (bulk copy) while these loads went through the
                // generic proxy: the proxy fence orders them before the refill that this arrival allows.
                fence_proxy_async_smem();
                mbar_arrive(bar(kDqBarDEmpty + st));
                ++unit;
            };
            auto load_row_f32 = [&](float (&dst)[64], int smem_off, int half) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4*>(smem + smem_off + swz_chunk_offset(r, half * 8 + c));
                    dst[8 * c + 0] = bf16_lo_to_f32(v.x); dst[8 * c + 1] = bf16_hi_to_f32(v.x);
                    dst[8 * c + 2] = bf16_lo_to_f32(v.y); dst[8 * c + 3] = bf16_hi_to_f32(v.y);
                    dst[8 * c + 4] = bf16_lo_to_f32(v.z); dst[8 * c + 5] = bf16_hi_to_f32(v.z);
                    dst[8 * c + 6] = bf16_lo_to_f32(v.w); dst[8 * c + 7] = bf16_hi_to_f32(v.w);
                }
            };
            auto dot64 = [&](const float (&x)[64], const uint4 (&y)[8]) {
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    a0 = fmaf(x[8 * c + 0], bf16_lo_to_f32(y[c].x), a0);
                    a1 = fmaf(x[8 * c + 1], bf16_hi_to_f32(y[c].x), a1);
                    a2 = fmaf(x[8 * c + 2], bf16_lo_to_f32(y[c].y), a2);
                    a3 = fmaf(x[8 * c + 3], bf16_hi_to_f32(y[c].y), a3);
                    a0 = fmaf(x[8 * c + 4], bf16_lo_to_f32(y[c].z), a0);
                    a1 = fmaf(x[8 * c + 5], bf16_hi_to_f32(y[c].z), a1);
                    a2 = fmaf(x[8 * c + 6], bf16_lo_to_f32(y[c].w), a2);
                    a3 = fmaf(x[8 * c + 7], bf16_hi_to_f32(y[c].w), a3);
                }
                return (a0 + a1) + (a2 + a3);
            };

#pragma unroll 1
            for (int g0 = 0; g0 < p.l; g0 += kDepthGroup) {
                const int gl = min(kDepthGroup, p.l - g0);
                // ---- pass A: u_i = <q, kd_i> ----
#pragma unroll 1
                for (int half = 0; half < NSUB; ++half) {
                    float q[64];
                    load_row_f32(q, L::kQ, half);
#pragma unroll 1
                    for (int ii = 0; ii < gl; ++ii) {
                        uint4 cur[8];
                        take_unit(cur);
                        const float part = dot64(q, cur);
                        if (half == 0) sU[ii * kTileRows + r] = part;
                        else sU[ii * kTileRows + r] += part;
                    }
                }
                // R_i = exp(u_i - LSE): the forward's LSE already covers sequence and depth keys.
                for (int ii = 0; ii < gl; ++ii)
                    sU[ii * kTileRows + r] = fast_exp2(fmaf(sU[ii * kTileRows + r], p.scale_log2, neg_lse2));

                // ---- pass B: <dO, vd_i>, and dVd_i = R_i dO ----
#pragma unroll 1
                for (int half = 0; half < NSUB; ++half) {
                    float g[64];
                    load_row_f32(g, L::kdO, half);
#pragma unroll 1
                    for (int ii = 0; ii < gl; ++ii) {
                        uint4 cur[8];
                        take_unit(cur);
                        const float part = dot64(g, cur);
                        if (half == 0) sDr[ii * kTileRows + r] = part;
                        else sDr[ii * kTileRows + r] += part;
                        if (store_grads) {
                            const float w = sU[ii * kTileRows + r];
                            uint4* dst = gV + size_t(g0 + ii) * slot_stride + (half * 8) * kTileRows;
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                uint4 o;
                                o.x = pack_bf16x2(w * g[8 * c + 0], w * g[8 * c + 1]);
                                o.y = pack_bf16x2(w * g[8 * c + 2], w * g[8 * c + 3]);
                                o.z = pack_bf16x2(w * g[8 * c + 4], w * g[8 * c + 5]);
                                o.w = pack_bf16x2(w * g[8 * c + 6], w * g[8 * c + 7]);
                                if (accumulate) red_add_bf16x2_v4(dst + c * kTileRows, o);
                                else dst[c * kTileRows] = o;
                            }
                        }
                    }
                }
                // dU_i = R_i (<dO, vd_i> - D)
                for (int ii = 0; ii < gl; ++ii)
                    sDr[ii * kTileRows + r] = sU[ii * kTileRows + r] * (sDr[ii * kTileRows + r] - delta);
                if (!store_grads) {
                    for (int ii = 0; ii < gl; ++ii) {
                        float* dst = rt_row + size_t(g0 + ii) * 2 * (kTileRows * p.G);
                        dst[0] = sU[ii * kTileRows + r];
                        dst[kTileRows * p.G] = sDr[ii * kTileRows + r];
                    }
                }

                // ---- pass C: dQ share sum_i dU_i kd_i (accumulated in TMEM across groups), dKd_i = scale dU_i q ----
#pragma unroll 1
                for (int half = 0; half < NSUB; ++half) {
                    uint4 qp[8];                           // q kept packed: only multiplied, never summed
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        qp[c] = *reinterpret_cast<const uint4*>(smem + L::kQ + swz_chunk_offset(r, half * 8 + c));
                    float acc[64];
                    if (g0 == 0) {
#pragma unroll
                        for (int c = 0; c < 64; ++c) acc[c] = 0.f;
                    } else {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tmem + lane_addr + kColdQd + half * 64 + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[32 * c + i] = __uint_as_float(o[i]);
                        }
                    }
#pragma unroll 1
                    for (int ii = 0; ii < gl; ++ii) {
                        uint4 cur[8];
                        take_unit(cur);
                        const float du = sDr[ii * kTileRows + r];
                        const float sdu = du * p.scale;
                        const uint32_t sdu2 = pack_bf16x2(sdu, sdu);
                        uint4* dst = gK + size_t(g0 + ii) * slot_stride + (half * 8) * kTileRows;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            acc[8 * c + 0] = fmaf(du, bf16_lo_to_f32(cur[c].x), acc[8 * c + 0]);
                            acc[8 * c + 1] = fmaf(du, bf16_hi_to_f32(cur[c].x), acc[8 * c + 1]);
                            acc[8 * c + 2] = fmaf(du, bf16_lo_to_f32(cur[c].y), acc[8 * c + 2]);
                            acc[8 * c + 3] = fmaf(du, bf16_hi_to_f32(cur[c].y), acc[8 * c + 3]);
                            acc[8 * c + 4] = fmaf(du, bf16_lo_to_f32(cur[c].z), acc[8 * c + 4]);
                            acc[8 * c + 5] = fmaf(du, bf16_hi_to_f32(cur[c].z), acc[8 * c + 5]);
                            acc[8 * c + 6] = fmaf(du, bf16_lo_to_f32(cur[c].w), acc[8 * c + 6]);
                            acc[8 * c + 7] = fmaf(du, bf16_hi_to_f32(cur[c].w), acc[8 * c + 7]);
                            uint4 o;
                            o.x = mul_bf16x2(qp[c].x, sdu2);
                            o.y = mul_bf16x2(qp[c].y, sdu2);
                            o.z = mul_bf16x2(qp[c].z, sdu2);
                            o.w = mul_bf16x2(qp[c].w, sdu2);
                            if (store_grads) {
                                if (accumulate) red_add_bf16x2_v4(dst + c * kTileRows, o);
                                else dst[c * kTileRows] = o;
                            }
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(acc[32 * c + i]);
                        tmem_st32(tmem + lane_addr + kColdQd + half * 64 + c * 32, o);
                    }
                    tmem_wait_st();                        // the next group reads these columns back
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(kDqBarDepth));
        }
    } else if (warp < 16) {
        setmaxnreg_dec<48>();
        if (warp == 12) {
            // =========================== TMA producer ===========================
            if (lane == 0) {
                tma_prefetch_desc(&mapQ);
                tma_prefetch_desc(&mapdO);
                tma_prefetch_desc(&mapK64);
                tma_prefetch_desc(&mapV64);
                mbar_arrive_expect_tx(bar(kDqBarQ), 2 * L::kTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s) {
                    tma_load_4d(sbase + L::kQ + s * L::kSubBytes, &mapQ, bar(kDqBarQ), s * 64, h, q0, b);
                    tma_load_4d(sbase + L::kdO + s * L::kSubBytes, &mapdO, bar(kDqBarQ), s * 64, h, q0, b);
                }
                for (int j = 0; j < n_kv; ++j) {
                    const int st = j % L::kStages;
                    if (j >= L::kStages)
                        mbar_wait(bar(kDqBarKVEmpty + st), ((j - L::kStages) / L::kStages) & 1, abort_flag, 70);
                    mbar_arrive_expect_tx(bar(kDqBarKVFull + st), 2 * L::kHalfTileBytes);
                    const uint32_t dstK = sbase + L::kKV + st * 2 * L::kHalfTileBytes;
                    const uint32_t dstV = dstK + L::kHalfTileBytes;
#pragma unroll
                    for (int s = 0; s < NSUB; ++s) {
                        tma_load_4d(dstK + s * L::kHalfSubBytes, &mapK64, bar(kDqBarKVFull + st), s * 64, hk, j * kKeyTile, b);
                        tma_load_4d(dstV + s * L::kHalfSubBytes, &mapV64, bar(kDqBarKVFull + st), s * 64, hk, j * kKeyTile, b);
                    }
                }
            }
        } else if (warp == 13) {
            // =========================== depth-cache producer ===========================
            // 16 KiB units in the order the depth warps consume them, group by group: keys (pass A),
            // values (pass B), keys again (pass C).
            if (lane == 0 && p.l > 0) {
                const uint64_t policy = l2_policy_evict_first();
                const size_t slot_bytes = cache_slot_elems(p.B, p.T, Hk, D) * 2;
                const size_t kv_bytes = size_t(kTileRows) * D * 2;
                const uint8_t* blk = reinterpret_cast<const uint8_t*>(p.depth_kv) +
                                     (((size_t(b) * Hk + hk) * nq + qt) * 2) * kv_bytes;
                // keys of a group are fetched twice; the first fetch is kept in L2 (evict_last), the second
                // fetch and the values are not needed again (evict_first)
                const uint64_t keep = l2_policy_evict_last();
                int unit = 0;
                for (int g0 = 0; g0 < p.l; g0 += kDepthGroup) {
                    const int gl = min(kDepthGroup, p.l - g0);
                    for (int pass = 0; pass < 3; ++pass) {
                        const int kv = (pass == 1) ? 1 : 0;
                        for (int half = 0; half < NSUB; ++half)
                            for (int ii = 0; ii < gl; ++ii, ++unit) {
                                const int st = unit % L::kRingStages;
                                if (unit >= L::kRingStages)
                                    mbar_wait(bar(kDqBarDEmpty + st), ((unit / L::kRingStages) - 1) & 1, abort_flag, 71);
                                mbar_arrive_expect_tx(bar(kDqBarDFull + st), L::kUnitBytes);
                                bulk_load(sbase + L::kRing + st * L::kUnitBytes,
                                          blk + size_t(g0 + ii) * slot_bytes + size_t(kv) * kv_bytes + size_t(half) * L::kUnitBytes,
                                          L::kUnitBytes, bar(kDqBarDFull + st), pass == 0 ? keep : policy);
                            }
                    }
                }
            }
        }
    } else {
        setmaxnreg_dec<48>();
        if (warp == 16 || warp == 17) {
            // ============ MMA issuers: S = Q K^T (warp 16), dP = dO V^T (warp 17) ============
            {   // whole warp: operands are warp-uniform, one elected lane issues
                const bool is_s = (warp == 16);
                constexpr uint32_t idesc_s = make_idesc_bf16(128, kKeyTile, false, false);
                const uint32_t a_tile = sbase + (is_s ? L::kQ : L::kdO);
                const uint32_t col = is_s ? kColS : kColdP;
                uint64_t da[D / 16];
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) da[kk] = desc_kmajor_sw128(a_tile + (kk >> 2) * L::kSubBytes, kk & 3);
                const uint64_t db0 = desc_kmajor_sw128(sbase + L::kKV + (is_s ? 0 : L::kHalfTileBytes), 0);
                mbar_wait(bar(kDqBarQ), 0, abort_flag, 81);
                for (int j = 0; j < n_kv; ++j) {
                    const int st = j % L::kStages, buf = j & 1;
                    if (j >= 2) {
                        // S buffer: dS_{j-2} overlays it until dQ_{j-2} has completed;
                        // dP buffer: free once the row warps have read dP_{j-2} (their arrival for tile j-2)
                        const uint32_t free_bar = is_s ? bar(kDqBarKVEmpty + (j - 2) % L::kStages) : bar(kDqBarPFull + buf);
                        const uint32_t free_par = is_s ? ((j - 2) / L::kStages) & 1 : ((j - 2) >> 1) & 1;
                        mbar_wait2(bar(kDqBarKVFull + st), (j / L::kStages) & 1, free_bar, free_par, abort_flag, 80, is_s ? 83 : 84);
                    } else {
                        mbar_wait(bar(kDqBarKVFull + st), (j / L::kStages) & 1, abort_flag, 80);
                    }
                    tc_fence_after_sync();
                    const uint64_t db = db0 + uint64_t((st * 2 * L::kHalfTileBytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        umma_ss(tmem + col + buf * 64, da[kk], db + uint64_t(((kk >> 2) * L::kHalfSubBytes + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                    umma_commit(bar(kDqBarSFull + buf));
                }
                drain_on_abort(is_s ? 0 : 1);
            }
        } else if (warp == 18) {
            // ============ MMA issuer: dQ += dS K (warp 18) ============
            {   // whole warp: operands are warp-uniform, one elected lane issues
                constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, false, true);
                const uint64_t db0 = desc_mnmajor_sw128(sbase + L::kKV, 0, L::kHalfSubBytes);
                for (int j = 0; j < n_kv; ++j) {
                    const int st = j % L::kStages, buf = j & 1;
                    mbar_wait(bar(kDqBarPFull + buf), (j >> 1) & 1, abort_flag, 82);
                    tc_fence_after_sync();
                    const uint64_t db = db0 + uint64_t((st * 2 * L::kHalfTileBytes) >> 4);
                    umma_ts(tmem + kColdQ, tmem + kColS + buf * 64, db, idesc_dq, j > 0);
#pragma unroll
                    for (int kk = 1; kk < kKeyTile / 16; ++kk)   // 16 keys per k-step: 8 columns, in block kk / 2
                        umma_ts(tmem + kColdQ, tmem + kColS + buf * 64 + (kk >> 1) * 32 + (kk & 1) * 8, db + uint64_t(kk * 128), idesc_dq, 1);
                    umma_commit(bar(kDqBarKVEmpty + st));
                }
                umma_commit(bar(kDqBarFinal));
                drain_on_abort(2);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag != 0 && tid == 256) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) {}
    }
    __syncthreads();
    if (warp == 16) tmem_dealloc(tmem, kTmemCols);
}

// =====================================================================================
// Depth gradients of a grouped-query backward
// =====================================================================================
// dKd_i[t] = scale sum_g dU_i^g[t] q^g[t] and dVd_i[t] = sum_g R_i^g[t] dO^g[t] over the G query heads
// of a key/value head, from the factors the dQ kernel left in the workspace.  Row-local and bound by
// the one write of the depth gradients: no depth cache is read.  A thread keeps FW features of the G
// rows (q^g or dO^g) in registers (G x FW = 64 values: FW = 8 up to G = 8, 4 at G = 16, 2 at G = 32) and
// walks the slots, writing FW bf16 per slot in cache layout (consecutive lanes = consecutive rows).
// One CTA = 128 rows x 4 feature pieces of one (b, hk, tile, dKd or dVd).  The factors of a few slots
// at a time are staged in shared memory (every thread of a row needs the same G factors per slot).
constexpr int kGroupGradThreads = 512;

template <int G>
struct GroupGrad {
    static_assert(G >= 2 && (G <= 8 || G == 16 || G == 32), "group size not supported");
    static constexpr int kFW = G <= 8 ? 8 : (G == 16 ? 4 : 2);      // features per thread
    static constexpr int kSlots = G <= 8 ? 8 : (G == 16 ? 4 : 2);   // slots staged at a time (<= 32 KiB)
};

template <int D, int G>
__global__ void __launch_bounds__(kGroupGradThreads)
depth_grad_group_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ dO,
                        const float* __restrict__ rowterms, __nv_bfloat16* __restrict__ d_depth_kv,
                        int B, int T, int Hk, int l, float scale, int accumulate) {
    constexpr int FW = GroupGrad<G>::kFW, SLOTS = GroupGrad<G>::kSlots;
    constexpr int PIECES = D / FW;                       // feature pieces per row
    constexpr int PGROUPS = PIECES / 4;                  // CTAs per (tile, kv)
    __shared__ __align__(16) float s_coef[SLOTS * kTileRows * G];
    const int nq = num_tiles(T);
    const int pgrp = blockIdx.x % PGROUPS;
    const int kv = (blockIdx.x / PGROUPS) & 1;           // 0: dKd (dU, q, scaled), 1: dVd (R, dO)
    const int tile_id = blockIdx.x / (2 * PGROUPS);      // (b * Hk + hk) * nq + qt
    const int qt = tile_id % nq;
    const int bhk = tile_id / nq;
    const int b = bhk / Hk, hk = bhk % Hk;
    const int r = threadIdx.x & 127;
    const int piece = pgrp * 4 + (threadIdx.x >> 7);     // features [piece * FW, piece * FW + FW)
    const int t = qt * kTileRows + r;
    const int H = Hk * G;
    const __nv_bfloat16* X = kv == 0 ? Q : dO;
    const float mul = kv == 0 ? scale : 1.f;
    float x[G][FW];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        uint32_t w[FW / 2];
#pragma unroll
        for (int k = 0; k < FW / 2; ++k) w[k] = 0u;      // rows past T contribute zeros: the tail stays zero
        if (t < T) {
            const __nv_bfloat16* src = X + ((size_t(b) * T + t) * H + hk * G + g) * D + piece * FW;
            if constexpr (FW == 8) {
                const uint4 v = *reinterpret_cast<const uint4*>(src);
                w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
            } else if constexpr (FW == 4) {
                const uint2 v = *reinterpret_cast<const uint2*>(src);
                w[0] = v.x; w[1] = v.y;
            } else {
                w[0] = *reinterpret_cast<const uint32_t*>(src);
            }
        }
#pragma unroll
        for (int k = 0; k < FW / 2; ++k) {
            x[g][2 * k] = bf16_lo_to_f32(w[k]) * mul;
            x[g][2 * k + 1] = bf16_hi_to_f32(w[k]) * mul;
        }
    }
    // factors of this tile: [slot][{R, dU}][g][row 128]; dKd uses dU, dVd uses R
    const float* coef = rowterms + (size_t(tile_id) * l * 2 + (kv == 0 ? 1 : 0)) * (kTileRows * G);
    const size_t slot_elems = cache_slot_elems(B, T, Hk, D);
    // cache block of (tile, kv): [chunk][row 128][8]; this thread's FW features sit inside one chunk
    __nv_bfloat16* out = d_depth_kv + (size_t(tile_id) * 2 + kv) * (kTileRows * D)
                         + (size_t((piece * FW) / 8) * kTileRows + r) * 8 + (piece * FW) % 8;
    for (int i0 = 0; i0 < l; i0 += SLOTS) {
        const int n = min(SLOTS, l - i0);
        __syncthreads();
        for (int e = threadIdx.x; e < n * kTileRows * G; e += kGroupGradThreads) {
            const int i = e / (kTileRows * G);
            s_coef[e] = coef[size_t(i0 + i) * 2 * (kTileRows * G) + (e - i * (kTileRows * G))];
        }
        __syncthreads();
        for (int i = 0; i < n; ++i) {
            float a[FW];
#pragma unroll
            for (int k = 0; k < FW; ++k) a[k] = 0.f;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float w = s_coef[(i * G + g) * kTileRows + r];
#pragma unroll
                for (int k = 0; k < FW; ++k) a[k] = fmaf(w, x[g][k], a[k]);
            }
            __nv_bfloat16* dst = out + size_t(i0 + i) * slot_elems;
            if constexpr (FW == 8) {
                uint4 o;
                o.x = pack_bf16x2(a[0], a[1]); o.y = pack_bf16x2(a[2], a[3]);
                o.z = pack_bf16x2(a[4], a[5]); o.w = pack_bf16x2(a[6], a[7]);
                if (accumulate) red_add_bf16x2_v4(dst, o);
                else *reinterpret_cast<uint4*>(dst) = o;
            } else if constexpr (FW == 4) {
                uint2 o;
                o.x = pack_bf16x2(a[0], a[1]); o.y = pack_bf16x2(a[2], a[3]);
                if (accumulate) red_add_bf16x2_v2(dst, o);
                else *reinterpret_cast<uint2*>(dst) = o;
            } else {
                if (accumulate) red_add_bf16x2(dst, pack_bf16x2(a[0], a[1]));
                else *reinterpret_cast<uint32_t*>(dst) = pack_bf16x2(a[0], a[1]);
            }
        }
    }
}

// =====================================================================================
// dK, dV
// =====================================================================================
// 512 threads.  Warps 0-3 and 4-7 form P^T / dS^T (each warpgroup takes 32 of the 64 query columns
// of an iteration; a thread owns one key row) and run the epilogue (dK by the first, dV by the
// second).  Warp 8 loads.  The four contractions of an iteration are issued by four threads on four
// schedulers, because one tcgen05.mma costs its issuing thread about 60 cycles: warp 9 S^T = K Q^T,
// warp 10 dP^T = V dO^T, warp 11 dV += P^T dO, warp 12 dK += dS^T Q.  MMAs of different threads are
// ordered by mbarriers only.
constexpr int kBwdDkvThreads = 512;

template <int D>
struct DkvSmem {
    static constexpr int kTileBytes = kTileRows * D * 2;
    static constexpr int kSubBytes = kTileRows * 128;
    static constexpr int kHalfTileBytes = kKeyTile * D * 2;
    static constexpr int kHalfSubBytes = kKeyTile * 128;
    static constexpr int kStages = 3;
    static constexpr int kK = 0;
    static constexpr int kV = kK + kTileBytes;
    static constexpr int kQdO = kV + kTileBytes;                       // stages of [Q_i | dO_i]
    // per stage, per pair of query columns: {-LSE c, -LSE c+1, D c, D c+1} (one 16-byte load per pair)
    static constexpr int kRowTerms = kQdO + kStages * 2 * kHalfTileBytes;
    static constexpr int kBars = kRowTerms + kStages * kKeyTile * 8;
    static constexpr int kNumBars = 16;
    static constexpr int kMisc = kBars + kNumBars * 8;
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
};

enum DkvBar : int {
    kDkvBarKV = 0,
    kDkvBarQFull = 1,    // +stage (3): Q_i, dO_i, LSE, D_t of the stage have landed
    kDkvBarQEmpty = 4,   // +stage (3), count 2: dV and dK of the stage's iteration are complete
    kDkvBarSFull = 7,    // +buffer (2), count 2: S^T and dP^T of the iteration are complete
    kDkvBarPFull = 9,    // +buffer (2), count 256: P^T and dS^T are written
    kDkvBarFinal = 11,   // count 2: the last dV and dK are complete
    kDkvBarDrain = 12,   // +issuer (4): abort path only
};

struct DkvParams {
    const float* LSE;
    const float* delta;
    int B, T, H;        // H = number of query heads
    int G;              // query heads per key/value head; dK, dV sum over the G heads of a group
    float scale, scale_log2;
};

template <int D>
__global__ void __launch_bounds__(kBwdDkvThreads, 1)
moda_bwd_dkdv_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                     const __grid_constant__ CUtensorMap mapQ64, const __grid_constant__ CUtensorMap mapdO64,
                     const __grid_constant__ CUtensorMap mapdK, const __grid_constant__ CUtensorMap mapdV,
                     const DkvParams p) {
    using L = DkvSmem<D>;
    constexpr int NSUB = D / 64;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColST = 0, kColdPT = 128, kColdK = 256, kColdV = 384;

    if (g_moda_status != 0) return;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    float4* sRow = reinterpret_cast<float4*>(smem + L::kRowTerms);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar = [&](int i) { return sbase + L::kBars + 8u * uint32_t(i); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nk = num_tiles(p.T);
    const int bh = blockIdx.x / nk;
    const int kt = blockIdx.x % nk;                       // key tiles in ascending order: most work first
    const int Hk = p.H / p.G;
    const int b = bh / Hk, h = bh % Hk;                   // h: key/value head of this CTA
    const int k0 = kt * kTileRows;
    const int nq64 = (p.T + kKeyTile - 1) / kKeyTile;
    const int i_first = 2 * kt;                           // first 64-query tile that can see this key tile
    const int n_per = nq64 - i_first;                     // query tiles per query head
    const int n_it = n_per * p.G;                         // iteration it: query head h G + it / n_per, tile i_first + it % n_per

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(kDkvBarKV), 1);
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar(kDkvBarQFull + s), 32);
            mbar_init(bar(kDkvBarQEmpty + s), 2);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kDkvBarSFull + s), 2);
            mbar_init(bar(kDkvBarPFull + s), 256);
        }
        mbar_init(bar(kDkvBarFinal), 2);
        for (int s = 0; s < 4; ++s) mbar_init(bar(kDkvBarDrain + s), 1);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Abort path of an issuing thread: wait (bounded) until its own MMAs have drained.
    auto drain_on_abort = [&](int which) {
        if (*abort_flag != 0) {
            umma_commit(bar(kDkvBarDrain + which));
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(bar(kDkvBarDrain + which), 0) && globaltimer_ns() - t0 < 20000000ull) {}
        }
    };

    if (warp < 8) {
        // =========================== P^T, dS^T and the dK / dV epilogue ===========================
        setmaxnreg_inc<152>();
        const int hc = warp >> 2;                            // which 32 query columns of every iteration
        const int r = tid & 127;                             // key row inside the tile = TMEM lane
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        for (int it = 0; it < n_it; ++it) {
            const int st = it % L::kStages, buf = it & 1;
            const int qoff = (i_first + it % n_per) * kKeyTile - k0;  // query of column c sees key row r iff qoff + c >= r
            mbar_wait(bar(kDkvBarQFull + st), (it / L::kStages) & 1, abort_flag, 90);   // LSE / D_t of this stage
            mbar_wait(bar(kDkvBarSFull + buf), (it >> 1) & 1, abort_flag, 91);
            tc_fence_after_sync();
            const float4* rt = sRow + st * (kKeyTile / 2) + hc * 16;
            const bool masked = qoff < kTileRows - 1;
            uint32_t s[32], g[32];
            tmem_ld32(tmem + lane_addr + kColST + buf * 64 + hc * 32, s);
            tmem_ld32(tmem + lane_addr + kColdPT + buf * 64 + hc * 32, g);
            tmem_wait_ld();
            // P^T overlays S^T, dS^T overlays dP^T (bf16, two per column).  Each warpgroup writes over
            // the first 16 of the 32 columns it has just read itself (columns 32 hc .. 32 hc + 15), so
            // the two never touch each other's scores; the MMA issuers address the two blocks per k-step.
            // Stored in two halves so that the first half's stores run under the second half's arithmetic.
            uint32_t pp[16], pd[16];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                for (int i = 8 * hh; i < 8 * hh + 8; ++i) {
                    const int c0 = hc * 32 + 2 * i;
                    const float4 t = rt[i];                  // {-LSE c0, -LSE c0+1, D c0, D c0+1}, same for all rows
                    float pa = fast_exp2(fmaf(__uint_as_float(s[2 * i]), p.scale_log2, t.x));
                    float pb = fast_exp2(fmaf(__uint_as_float(s[2 * i + 1]), p.scale_log2, t.y));
                    if (masked) {
                        if (qoff + c0 < r) pa = 0.f;
                        if (qoff + c0 + 1 < r) pb = 0.f;
                    }
                    pp[i] = pack_bf16x2(pa, pb);
                    pd[i] = pack_bf16x2(pa * (__uint_as_float(g[2 * i]) - t.z), pb * (__uint_as_float(g[2 * i + 1]) - t.w));
                }
                tmem_st8(tmem + lane_addr + kColST + buf * 64 + hc * 32 + 8 * hh, pp + 8 * hh);
                tmem_st8(tmem + lane_addr + kColdPT + buf * 64 + hc * 32 + 8 * hh, pd + 8 * hh);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(kDkvBarPFull + buf));
        }
        mbar_wait(bar(kDkvBarFinal), 0, abort_flag, 92);
        tc_fence_after_sync();
        {                                                    // first warpgroup: dK (scaled); second: dV
            const float mul = hc == 0 ? p.scale : 1.f;
            const uint32_t col = hc == 0 ? kColdK : kColdV;
            const int dst_off = hc == 0 ? L::kK : L::kV;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tmem + lane_addr + col + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int g4 = 0; g4 < 4; ++g4) {
                    uint4 v;
                    v.x = pack_bf16x2(__uint_as_float(o[8 * g4 + 0]) * mul, __uint_as_float(o[8 * g4 + 1]) * mul);
                    v.y = pack_bf16x2(__uint_as_float(o[8 * g4 + 2]) * mul, __uint_as_float(o[8 * g4 + 3]) * mul);
                    v.z = pack_bf16x2(__uint_as_float(o[8 * g4 + 4]) * mul, __uint_as_float(o[8 * g4 + 5]) * mul);
                    v.w = pack_bf16x2(__uint_as_float(o[8 * g4 + 6]) * mul, __uint_as_float(o[8 * g4 + 7]) * mul);
                    *reinterpret_cast<uint4*>(smem + dst_off + swz_chunk_offset(r, c * 4 + g4)) = v;
                }
            }
        }
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0) {
#pragma unroll
            for (int s = 0; s < NSUB; ++s) {
                tma_store_4d(&mapdK, sbase + L::kK + s * L::kSubBytes, s * 64, h, k0, b);
                tma_store_4d(&mapdV, sbase + L::kV + s * L::kSubBytes, s * 64, h, k0, b);
            }
            tma_store_commit();
            tma_store_wait_all();
        }
    } else if (warp < 12) {
      setmaxnreg_dec<64>();
      if (warp == 8) {
        // =========================== loader: TMA tiles + per-query LSE, D_t ===========================
        if (lane == 0) {
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            tma_prefetch_desc(&mapQ64);
            tma_prefetch_desc(&mapdO64);
            mbar_arrive_expect_tx(bar(kDkvBarKV), 2 * L::kTileBytes);
#pragma unroll
            for (int s = 0; s < NSUB; ++s) {
                tma_load_4d(sbase + L::kK + s * L::kSubBytes, &mapK, bar(kDkvBarKV), s * 64, h, k0, b);
                tma_load_4d(sbase + L::kV + s * L::kSubBytes, &mapV, bar(kDkvBarKV), s * 64, h, k0, b);
            }
        }
        for (int it = 0; it < n_it; ++it) {
            const int st = it % L::kStages;
            const int hq = h * p.G + it / n_per;
            const size_t row_base = (size_t(b) * p.H + hq) * p.T;
            const int qrow0 = (i_first + it % n_per) * kKeyTile;
            if (it >= L::kStages)
                mbar_wait(bar(kDkvBarQEmpty + st), ((it - L::kStages) / L::kStages) & 1, abort_flag, 100);
            {
                // lane handles the column pair (2 lane, 2 lane + 1); invalid (padding) queries get
                // -LSE = -inf so that their P is exactly 0
                const int c = 2 * lane;
                float4 t;
                t.x = (qrow0 + c < p.T) ? -p.LSE[row_base + qrow0 + c] * kLog2e : -INFINITY;
                t.y = (qrow0 + c + 1 < p.T) ? -p.LSE[row_base + qrow0 + c + 1] * kLog2e : -INFINITY;
                t.z = (qrow0 + c < p.T) ? p.delta[row_base + qrow0 + c] : 0.f;
                t.w = (qrow0 + c + 1 < p.T) ? p.delta[row_base + qrow0 + c + 1] : 0.f;
                sRow[st * (kKeyTile / 2) + lane] = t;
            }
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(kDkvBarQFull + st), 2 * L::kHalfTileBytes);
                const uint32_t dstQ = sbase + L::kQdO + st * 2 * L::kHalfTileBytes;
                const uint32_t dstdO = dstQ + L::kHalfTileBytes;
#pragma unroll
                for (int s = 0; s < NSUB; ++s) {
                    tma_load_4d(dstQ + s * L::kHalfSubBytes, &mapQ64, bar(kDkvBarQFull + st), s * 64, hq, qrow0, b);
                    tma_load_4d(dstdO + s * L::kHalfSubBytes, &mapdO64, bar(kDkvBarQFull + st), s * 64, hq, qrow0, b);
                }
            } else {
                mbar_arrive(bar(kDkvBarQFull + st));
            }
        }
      } else if (warp == 9 || warp == 10) {
        // ============ MMA issuers: S^T = K Q^T (warp 9), dP^T = V dO^T (warp 10) ============
        {   // whole warp: operands are warp-uniform, one elected lane issues
            const bool is_s = (warp == 9);
            constexpr uint32_t idesc_s = make_idesc_bf16(128, kKeyTile, false, false);
            const uint32_t a_tile = sbase + (is_s ? L::kK : L::kV);
            const uint32_t col = is_s ? kColST : kColdPT;
            uint64_t da[D / 16];
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) da[kk] = desc_kmajor_sw128(a_tile + (kk >> 2) * L::kSubBytes, kk & 3);
            const uint64_t db0 = desc_kmajor_sw128(sbase + L::kQdO + (is_s ? 0 : L::kHalfTileBytes), 0);
            mbar_wait(bar(kDkvBarKV), 0, abort_flag, 111);
            for (int it = 0; it < n_it; ++it) {
                const int st = it % L::kStages, buf = it & 1;
                mbar_wait(bar(kDkvBarQFull + st), (it / L::kStages) & 1, abort_flag, 110);
                // buffer `buf` still feeds dV / dK of iteration it-2 (P^T, dS^T overlay it)
                if (it >= 2) mbar_wait(bar(kDkvBarQEmpty + (it - 2) % L::kStages), ((it - 2) / L::kStages) & 1, abort_flag, 113);
                tc_fence_after_sync();
                const uint64_t db = db0 + uint64_t((st * 2 * L::kHalfTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    umma_ss(tmem + col + buf * 64, da[kk], db + uint64_t(((kk >> 2) * L::kHalfSubBytes + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                umma_commit(bar(kDkvBarSFull + buf));
            }
            drain_on_abort(is_s ? 0 : 1);
        }
      } else {
        // ============ MMA issuer: dV += P^T dO (warp 11) ============
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, false, true);
            const uint64_t db0 = desc_mnmajor_sw128(sbase + L::kQdO + L::kHalfTileBytes, 0, L::kHalfSubBytes);
            for (int it = 0; it < n_it; ++it) {
                const int st = it % L::kStages, buf = it & 1;
                mbar_wait(bar(kDkvBarPFull + buf), (it >> 1) & 1, abort_flag, 112);
                tc_fence_after_sync();
                const uint64_t db = db0 + uint64_t((st * 2 * L::kHalfTileBytes) >> 4);
                umma_ts(tmem + kColdV, tmem + kColST + buf * 64, db, idesc_acc, it > 0);
#pragma unroll
                for (int kk = 1; kk < kKeyTile / 16; ++kk)   // 16 queries per k-step: 8 columns, in block kk / 2
                    umma_ts(tmem + kColdV, tmem + kColST + buf * 64 + (kk >> 1) * 32 + (kk & 1) * 8, db + uint64_t(kk * 128), idesc_acc, 1);
                umma_commit(bar(kDkvBarQEmpty + st));
            }
            umma_commit(bar(kDkvBarFinal));
            drain_on_abort(2);
        }
      }
    } else {
      setmaxnreg_dec<64>();
      if (warp == 12) {
        // ============ MMA issuer: dK += dS^T Q (warp 12) ============
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, false, true);
            const uint64_t db0 = desc_mnmajor_sw128(sbase + L::kQdO, 0, L::kHalfSubBytes);
            for (int it = 0; it < n_it; ++it) {
                const int st = it % L::kStages, buf = it & 1;
                mbar_wait(bar(kDkvBarPFull + buf), (it >> 1) & 1, abort_flag, 114);
                tc_fence_after_sync();
                const uint64_t db = db0 + uint64_t((st * 2 * L::kHalfTileBytes) >> 4);
                umma_ts(tmem + kColdK, tmem + kColdPT + buf * 64, db, idesc_acc, it > 0);
#pragma unroll
                for (int kk = 1; kk < kKeyTile / 16; ++kk)
                    umma_ts(tmem + kColdK, tmem + kColdPT + buf * 64 + (kk >> 1) * 32 + (kk & 1) * 8, db + uint64_t(kk * 128), idesc_acc, 1);
                umma_commit(bar(kDkvBarQEmpty + st));
            }
            umma_commit(bar(kDkvBarFinal));
            drain_on_abort(3);
        }
      }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag != 0 && tid == 128) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) {}
    }
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace moda
