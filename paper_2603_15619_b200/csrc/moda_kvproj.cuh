// Key / value projection with the depth stream's write step in its epilogue (Sec. 2.1: K = X W_K, V = X W_V;
// Sec. 2.2, "write": a layer's key-value pair is appended to the depth stream, and an FFN layer obtains its pair
// through a KV projection of its input).
//
//   K[b, t, h, :] = X[b, t, :] Wk[h d : (h+1) d, :]^T        V likewise        (bf16 in, fp32 accumulation, bf16 out)
//
// One CTA owns one (b, 128-position tile) and NH key/value heads (two at d = 64 when H_k is even, else one): the
// output tile of a head is exactly one block of the depth cache (moda_cache.cuh), so the epilogue stores the rounded
// tile twice from the same registers: as the K / V tensors [B][T][H_k][d] (through shared memory and a TMA store) and
// as the cache slot's blocks (chunk c of row r to [c][r]: 512 contiguous bytes per warp store).  K and V share the X
// tiles: the Wk and Wv tiles of a stage are adjacent in shared memory and form one B operand of 2 NH d rows, so one
// tcgen05.mma (M 128, N 2 NH d <= 256, K 16) feeds both accumulators.
//
//   warp 0      TMA producer: per 64 input features one X tile [128 x 64] and one Wk and one Wv tile [NH d x 64]
//               through a ring (128-byte swizzle); two CTAs fit an SM, so one's epilogue runs under the other's loop
//   warp 1      MMA issuer (owns the tensor-memory allocation): 4 tcgen05.mma per stage
//   warps 2-5   epilogue: a thread owns one position (= TMEM lane)
#pragma once

#include "moda_cache.cuh"
#include "moda_fwd.cuh"          // swz_chunk_offset
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kProjThreads = 192;

#ifndef MODA_PROJ_STAGES
#define MODA_PROJ_STAGES 2
#endif
template <int D, int NH>
struct KvProjSmem {
    static constexpr int kStages = MODA_PROJ_STAGES;
    static constexpr int kNW = D * NH;                         // output features per W tile
    static constexpr int kXBytes = kTileRows * 128;            // 128 positions x 64 features bf16
    static constexpr int kWBytes = kNW * 128;                  // NH d output features x 64 input features bf16
    static constexpr int kStageBytes = kXBytes + 2 * kWBytes;
    static constexpr int kRing = 0;
    static constexpr int kOutBytes = 2 * kTileRows * kNW * 2;  // K and V tiles for the TMA stores, over the ring
    static_assert(kOutBytes <= kStages * kStageBytes, "output staging does not fit the ring");
    static constexpr int kBars = kStages * kStageBytes;        // full[4], empty[4], accumulators complete
    static constexpr int kMisc = kBars + 16 * 8;               // tmem base, abort flag
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;             // slack for aligning the segment by hand
};

struct KvProjParams {
    __nv_bfloat16* slot;       // base of the cache slot to write (row-interleaved layout, H_k heads), or null
    int B, T, Hk, Dm;          // Dm = input features (a multiple of 64)
    int store_kv;              // nonzero: K and V are also stored as [B][T][H_k][d] tensors
};

template <int D, int NH>
__global__ void __launch_bounds__(kProjThreads, 2)
moda_kv_project_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapWk,
                       const __grid_constant__ CUtensorMap mapWv, const __grid_constant__ CUtensorMap mapK,
                       const __grid_constant__ CUtensorMap mapV, const KvProjParams p) {
    using L = KvProjSmem<D, NH>;
    constexpr int NSUB = D / 64;
    constexpr int NW = L::kNW;
    constexpr uint32_t kTmemCols = 2 * NW;                     // 128 or 256: K accumulators of the NH heads, then V
    if (g_moda_status != 0) return;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = aligned_dynamic_smem(smem_raw, L::kTotal);
    if (smem == nullptr) {
        if (threadIdx.x == 0) atomicCAS(&g_moda_status, 0, kStatusSmemLayout);
        return;
    }
    const uint32_t sbase = smem_u32(smem);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar_full = [&](int s) { return sbase + L::kBars + 8u * uint32_t(s); };
    auto bar_empty = [&](int s) { return sbase + L::kBars + 8u * uint32_t(L::kStages + s); };
    const uint32_t bar_acc = sbase + L::kBars + 8u * uint32_t(2 * L::kStages);
    const uint32_t bar_drain = bar_acc + 8u;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nt = num_tiles(p.T);
    const int hgroups = p.Hk / NH;
    const int hk0 = (blockIdx.x % hgroups) * NH;               // first of this CTA's heads
    const int tile = (blockIdx.x / hgroups) % nt;
    const int b = blockIdx.x / (hgroups * nt);
    const int t0 = tile * kTileRows;
    const int n_k = p.Dm / 64;

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 1);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_drain, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            tma_prefetch_desc(&mapX);
            tma_prefetch_desc(&mapWk);
            tma_prefetch_desc(&mapWv);
            for (int k = 0; k < n_k; ++k) {
                const int st = k % L::kStages;
                if (k >= L::kStages) mbar_wait(bar_empty(st), ((k / L::kStages) - 1) & 1, abort_flag, 160);
                const uint32_t dst = sbase + L::kRing + st * L::kStageBytes;
                mbar_arrive_expect_tx(bar_full(st), L::kStageBytes);
                // the tensors are addressed as [outer][rows][Dm / 64][64]: coordinate 1 picks the 64 input features
                tma_load_4d(dst, &mapX, bar_full(st), 0, k, t0, b);
                tma_load_4d(dst + L::kXBytes, &mapWk, bar_full(st), 0, k, hk0 * D, 0);
                tma_load_4d(dst + L::kXBytes + L::kWBytes, &mapWv, bar_full(st), 0, k, hk0 * D, 0);
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        constexpr uint32_t idesc = make_idesc_bf16(128, 2 * NW, false, false);
        for (int k = 0; k < n_k; ++k) {
            const int st = k % L::kStages;
            mbar_wait(bar_full(st), (k / L::kStages) & 1, abort_flag, 161);
            tc_fence_after_sync();
            const uint32_t x = sbase + L::kRing + st * L::kStageBytes;
            // B = the Wk tile and, right behind it, the Wv tile: 2 NW rows of 128 bytes, 8-row groups 1024 bytes apart
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_ss(tmem, desc_kmajor_sw128(x, kk), desc_kmajor_sw128(x + L::kXBytes, kk), idesc, (k > 0 || kk > 0) ? 1u : 0u);
            umma_commit(bar_empty(st));
        }
        umma_commit(bar_acc);
        if (*abort_flag != 0) {
            // a wait gave up somewhere: make sure no MMA is still in flight before tensor memory is released
            umma_commit(bar_drain);
            const uint64_t t_start = globaltimer_ns();
            while (!mbar_try_wait(bar_drain, 0) && globaltimer_ns() - t_start < 20000000ull) {}
        }
    } else {
        // =========================== epilogue ===========================
        const int r = (warp & 3) * 32 + lane;                  // position inside the tile = TMEM lane of this warp's quadrant
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        mbar_wait(bar_acc, 0, abort_flag, 162);
        tc_fence_after_sync();
        // every MMA has completed, so the ring is free: it becomes the staging of the two output tiles
        constexpr int CH = D / 8;
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
#pragma unroll
            for (int j = 0; j < NH; ++j) {
                uint4* slot_blk = p.slot == nullptr ? nullptr
                                  : reinterpret_cast<uint4*>(p.slot) + (((size_t(b) * p.Hk + hk0 + j) * nt + tile) * 2 + kv) * (kTileRows * CH) + r;
                uint8_t* stage = smem + L::kRing + (kv * NH + j) * (kTileRows * D * 2);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t a[32];
                    tmem_ld32(tmem + lane_addr + kv * NW + j * D + c * 32, a);
                    tmem_wait_ld();
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(a[8 * g + 0]), __uint_as_float(a[8 * g + 1]));
                        v.y = pack_bf16x2(__uint_as_float(a[8 * g + 2]), __uint_as_float(a[8 * g + 3]));
                        v.z = pack_bf16x2(__uint_as_float(a[8 * g + 4]), __uint_as_float(a[8 * g + 5]));
                        v.w = pack_bf16x2(__uint_as_float(a[8 * g + 6]), __uint_as_float(a[8 * g + 7]));
                        const int chunk = c * 4 + g;
                        // rows past T were loaded as zeros: the cache wants exactly that in its tail rows
                        if (slot_blk != nullptr) slot_blk[chunk * kTileRows] = v;
                        if (p.store_kv) *reinterpret_cast<uint4*>(stage + swz_chunk_offset(r, chunk)) = v;
                    }
                }
            }
        }
        if (p.store_kv) {
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (tid == 64) {
#pragma unroll
                for (int j = 0; j < NH; ++j)
#pragma unroll
                    for (int s = 0; s < NSUB; ++s) {
                        tma_store_4d(&mapK, sbase + L::kRing + j * (kTileRows * D * 2) + s * (kTileRows * 128), s * 64, hk0 + j, t0, b);
                        tma_store_4d(&mapV, sbase + L::kRing + (NH + j) * (kTileRows * D * 2) + s * (kTileRows * 128), s * 64, hk0 + j, t0, b);
                    }
                tma_store_commit();
                tma_store_wait_all();
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag != 0 && tid == 0) {
        const uint64_t t_start = globaltimer_ns();
        while (globaltimer_ns() - t_start < 2000000ull) {}     // abort path only: let copies in flight land
    }
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace moda
