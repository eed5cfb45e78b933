// Key / value projection with the depth stream's write step in its epilogue (Sec. 2.1: K = X W_K, V = X W_V;
// Sec. 2.2, "write": a layer's key-value pair is appended to the depth stream, and an FFN layer obtains its pair
// through a KV projection of its input).
//
//   K[b, t, h, :] = X[b, t, :] Wk[h d : (h+1) d, :]^T        V likewise        (bf16 in, fp32 accumulation, bf16 out)
//
// The output tile of (128 positions, one key/value head) is exactly one block of the depth cache (moda_cache.cuh), so
// the epilogue stores the rounded tile twice from the same registers: as the K / V tensors [B][T][H_k][d] (through shared
// memory and TMA stores) and as the cache slot's blocks (chunk c of row r to [c][r]: 512 contiguous bytes per warp
// store).  K and V share the X tiles: the Wk and Wv rows of NH heads (two at d = 64 when H_k is even, else one) form one
// B operand of 2 NH d <= 256 rows, so one tensor-core instruction per 16 features feeds both accumulators.
//
// Persistent kernel on CTA pairs (clusters of two, cta_group::2), 192 threads per CTA:
//   warp 0      TMA producer (both CTAs): per 64 input features its own X tile [128 x 64] and its half of B [NH d x 64]
//   warp 1      MMA issuer (the even CTA's; both CTAs' warp 1 allocate and free tensor memory together)
//   warps 2-5   epilogue (both CTAs): a thread owns one position (= TMEM lane) of its CTA's 128
//
// A pair owns 256 positions (two adjacent tiles of one batch entry) and NH heads per work item and walks the items
// round-robin.  Each CTA loads its own X tile and HALF of the B operand (the even CTA the Wk rows, the odd one the Wv
// rows): 32 KiB per 64 features instead of the 48 a CTA on its own would need for the same instruction shape (such a
// kernel, two CTAs per SM, ran at 74 % of the tensor peak, at 90 % with its loads taken out).  The even CTA issues one tcgen05.mma.cta_group::2 (M 256, N 2 NH d, K 16) per 16 features; the accumulator rows of a
// CTA's own 128 positions land in its own tensor memory, columns [0, NW) = K, [NW, 2 NW) = V.  Two accumulator sets
// alternate between items, so the epilogue of one item (tensor memory -> cache blocks with plain stores, and -> K / V
// tiles through one 32 KiB staging buffer and TMA stores, K first, then V) runs under the main loop of the next; CTAs of
// equal length that merely share an SM would run their epilogues at the same time.  The rest of shared memory is the
// operand ring: its depth is what the rate depends on (3 / 4 / 5 stages: 75 / 81 / 83 % of the tensor peak), since a
// refill goes issuer -> commit -> other CTA's producer -> TMA -> even CTA's barrier.  (K / V rows stored straight from
// registers, 64 contiguous bytes per thread, would free the staging for a seventh stage but run slower: 80 %.)
//
// Barriers: full[st] lives in the even CTA and counts the bytes of both CTAs' loads (the odd CTA's loads name it as a
// cluster address); empty[st] and acc_full[set] exist in both CTAs and the issuer commits to each; acc_empty[set] lives
// in the even CTA and takes one arrival per epilogue warp of either CTA.  All waits are bounded; the cluster barrier at
// the end keeps either CTA's shared memory alive until both are done.
#pragma once

#include "moda_cache.cuh"
#include "moda_fwd.cuh"          // swz_chunk_offset
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kProjThreads = 192;

struct KvProjParams {
    void* slot;                // base of the cache slot to write (row-interleaved bf16 layout, or e4m3 codes + row scales; H_k heads), or null
    int B, T, Hk, Dm;          // Dm = input features (a multiple of 64)
    int store_kv;              // nonzero: K and V are also stored as [B][T][H_k][d] tensors
};

#ifndef MODA_PROJ_STAGES
#define MODA_PROJ_STAGES 6
#endif
template <int D, int NH>
struct KvProjSmem {
    static constexpr int kStages = MODA_PROJ_STAGES;
    static constexpr int kNW = D * NH;
    static constexpr int kXBytes = kTileRows * 128;
    static constexpr int kWBytes = kNW * 128;                  // this CTA's half of B: NW rows of Wk or of Wv
    static constexpr int kStageBytes = kXBytes + kWBytes;
    static constexpr int kRing = 0;
    static constexpr int kOut = kStages * kStageBytes;         // the K tiles, then the V tiles, of the NH heads for the TMA stores
    static constexpr int kOutBytes = kTileRows * kNW * 2;
    static constexpr int kBars = kOut + kOutBytes;             // full[S], empty[S], acc_full[2], acc_empty[2], drain
    static constexpr int kMisc = kBars + (2 * kStages + 5) * 8;
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static_assert(kDynamic <= 232448, "shared-memory plan does not fit");
};

// FP8: the slot is written in the e4m3 layout (moda_cache.cuh): a thread owns a whole row of a head, so it takes the
// row's largest magnitude (of the values rounded to bf16, which is what K and V are) in a first pass over its
// accumulator columns, then scale = max / 448 and the codes in a second pass: the arithmetic of depth_cache_quant_kernel.
template <int D, int NH, bool FP8 = false>
__global__ void __launch_bounds__(kProjThreads, 1)
moda_kv_project_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapWk,
                            const __grid_constant__ CUtensorMap mapWv, const __grid_constant__ CUtensorMap mapK,
                            const __grid_constant__ CUtensorMap mapV, const KvProjParams p) {
    using L = KvProjSmem<D, NH>;
    constexpr int NW = L::kNW;
    constexpr uint32_t kTmemCols = 4 * NW;                     // two accumulator sets of 2 NW columns
    // Both CTAs of a pair must take the same way to the cluster barriers, so nothing here depends on the status word
    // (which another kernel may set between the two CTAs' reads); the host refuses calls after a fault anyway.  The
    // alignment of the shared segment is the same in every CTA of the launch.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = aligned_dynamic_smem(smem_raw, L::kTotal);
    if (smem == nullptr) {
        if (threadIdx.x == 0) atomicCAS(&g_moda_status, 0, kStatusSmemLayout);
        return;
    }
    const uint32_t rank = cluster_cta_rank();
    const uint32_t sbase = smem_u32(smem);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar_full = [&](int s) { return sbase + L::kBars + 8u * uint32_t(s); };
    auto bar_empty = [&](int s) { return sbase + L::kBars + 8u * uint32_t(L::kStages + s); };
    auto bar_acc_full = [&](int s) { return sbase + L::kBars + 8u * uint32_t(2 * L::kStages + s); };
    auto bar_acc_empty = [&](int s) { return sbase + L::kBars + 8u * uint32_t(2 * L::kStages + 2 + s); };
    const uint32_t bar_drain = sbase + L::kBars + 8u * uint32_t(2 * L::kStages + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nt = num_tiles(p.T);
    const int npairs = (nt + 1) / 2;
    const int hgroups = p.Hk / NH;
    const int n_items = p.B * npairs * hgroups;
    const int n_clusters = int(gridDim.x >> 1);
    const int cl = blockIdx.x >> 1;
    const int n_k = p.Dm / 64;

    if (tid == 0) {
        // after a fault anywhere the waits below fall through at once (results are garbage, the host reports the fault)
        *abort_flag = g_moda_status != 0 ? 1 : 0;
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_acc_full(s), 1);
            mbar_init(bar_acc_empty(s), 8);                    // four epilogue warps in each CTA
        }
        mbar_init(bar_drain, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // =========================== TMA producer (both CTAs) ===========================
        if (lane == 0) {
            const CUtensorMap* mapW = rank == 0 ? &mapWk : &mapWv;
            tma_prefetch_desc(&mapX);
            tma_prefetch_desc(mapW);
            int n = 0;                                         // stages filled so far
            for (int item = cl; item < n_items; item += n_clusters) {
                const int hk0 = (item % hgroups) * NH;
                const int t0 = (((item / hgroups) % npairs) * 2 + int(rank)) * kTileRows;   // may lie past T: zeros
                const int b = item / (hgroups * npairs);
                for (int k = 0; k < n_k; ++k, ++n) {
                    const int st = n % L::kStages;
                    if (n >= L::kStages) mbar_wait(bar_empty(st), ((n / L::kStages) - 1) & 1, abort_flag, 163);
                    const uint32_t dst = sbase + L::kRing + st * L::kStageBytes;
                    if (rank == 0) {
                        mbar_arrive_expect_tx(bar_full(st), 2 * L::kStageBytes);
                        tma_load_4d(dst, &mapX, bar_full(st), 0, k, t0, b);
                        tma_load_4d(dst + L::kXBytes, mapW, bar_full(st), 0, k, hk0 * D, 0);
                    } else {
                        const uint32_t full0 = cluster_map_shared(bar_full(st), 0);
                        tma_load_4d_pair(dst, &mapX, full0, 0, k, t0, b);
                        tma_load_4d_pair(dst + L::kXBytes, mapW, full0, 0, k, hk0 * D, 0);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer (even CTA) ===========================
        if (rank == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, 2 * NW, false, false);
            int n = 0, i = 0;
            for (int item = cl; item < n_items; item += n_clusters, ++i) {
                const int set = i & 1;
                if (i >= 2) {
                    mbar_wait(bar_acc_empty(set), ((i >> 1) - 1) & 1, abort_flag, 166);
                    tc_fence_after_sync();
                }
                const uint32_t acc = tmem + uint32_t(set * 2 * NW);
                for (int k = 0; k < n_k; ++k, ++n) {
                    const int st = n % L::kStages;
                    mbar_wait(bar_full(st), (n / L::kStages) & 1, abort_flag, 164);
                    tc_fence_after_sync();
                    const uint32_t x = sbase + L::kRing + st * L::kStageBytes;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_ss_pair(acc, desc_kmajor_sw128(x, kk), desc_kmajor_sw128(x + L::kXBytes, kk), idesc, (k > 0 || kk > 0) ? 1u : 0u);
                    umma_commit_pair(bar_empty(st));
                    umma_commit_pair(cluster_map_shared(bar_empty(st), 1));
                }
                umma_commit_pair(bar_acc_full(set));
                umma_commit_pair(cluster_map_shared(bar_acc_full(set), 1));
            }
            if (*abort_flag != 0) {
                umma_commit_pair(bar_drain);
                const uint64_t t_start = globaltimer_ns();
                while (!mbar_try_wait(bar_drain, 0) && globaltimer_ns() - t_start < 20000000ull) {}
            }
        }
    } else {
        // =========================== epilogue (both CTAs, own 128 positions) ===========================
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        constexpr int CH = D / 8;
        int i = 0;
        for (int item = cl; item < n_items; item += n_clusters, ++i) {
            const int set = i & 1;
            const int hk0 = (item % hgroups) * NH;
            const int tile = ((item / hgroups) % npairs) * 2 + int(rank);
            const int b = item / (hgroups * npairs);
            const bool live = tile < nt;                       // the odd CTA of the last pair may have no tile
            mbar_wait(bar_acc_full(set), (i >> 1) & 1, abort_flag, 165);
            tc_fence_after_sync();
            const int t0 = tile * kTileRows;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                if (p.store_kv) {
                    // the staging buffer is free once the TMA stores issued from it have read it
                    if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                }
#pragma unroll
                for (int j = 0; j < NH; ++j) {
                    const size_t blk_index = ((size_t(b) * p.Hk + hk0 + j) * nt + tile) * 2 + kv;
                    uint4* slot_blk = (p.slot == nullptr || !live) ? nullptr
                                      : FP8 ? reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.slot) + blk_index * cache8_block_bytes(D)) + r
                                            : reinterpret_cast<uint4*>(p.slot) + blk_index * (kTileRows * CH) + r;
                    uint8_t* stage = smem + L::kOut + j * (kTileRows * D * 2);
                    float q_scale = 1.f;
                    RowDivider dv = make_row_divider(1.f);
                    if constexpr (FP8) {
                        float am = 0.f;
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t a[32];
                            tmem_ld32(tmem + lane_addr + set * 2 * NW + kv * NW + j * D + c * 32, a);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                const uint32_t w = pack_bf16x2(__uint_as_float(a[i]), __uint_as_float(a[i + 1]));
                                am = fmaxf(am, fmaxf(fabsf(bf16_lo_to_f32(w)), fabsf(bf16_hi_to_f32(w))));
                            }
                        }
                        q_scale = am > 0.f ? __fdiv_rn(am, 448.f) : 1.f;
                        dv = make_row_divider(q_scale);
                        if (slot_blk != nullptr)
                            reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(slot_blk - r) + size_t(kTileRows) * D)[r] = q_scale;
                    }
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t a[32];
                        tmem_ld32(tmem + lane_addr + set * 2 * NW + kv * NW + j * D + c * 32, a);
                        tmem_wait_ld();
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = pack_bf16x2(__uint_as_float(a[2 * i]), __uint_as_float(a[2 * i + 1]));
                        if constexpr (FP8) {
                            // 16 features per 16-byte chunk of codes
#pragma unroll
                            for (int g = 0; g < 2; ++g) {
                                uint32_t cw[4];
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const uint32_t w0 = w[8 * g + 2 * k], w1 = w[8 * g + 2 * k + 1];
                                    uint16_t lo, hi;
                                    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo)
                                        : "f"(div_rn(bf16_hi_to_f32(w0), dv)), "f"(div_rn(bf16_lo_to_f32(w0), dv)));
                                    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi)
                                        : "f"(div_rn(bf16_hi_to_f32(w1), dv)), "f"(div_rn(bf16_lo_to_f32(w1), dv)));
                                    cw[k] = uint32_t(lo) | (uint32_t(hi) << 16);
                                }
                                if (slot_blk != nullptr) slot_blk[(c * 2 + g) * kTileRows] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
                            }
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint4 v = make_uint4(w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
                            const int chunk = c * 4 + g;
                            // rows past T were loaded as zeros: the cache wants exactly that in its tail rows
                            if (!FP8 && slot_blk != nullptr) slot_blk[chunk * kTileRows] = v;
                            if (p.store_kv) *reinterpret_cast<uint4*>(stage + swz_chunk_offset(r, chunk)) = v;
                        }
                    }
                }
                if (p.store_kv) {
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (tid == 64 && live) {
#pragma unroll
                        for (int j = 0; j < NH; ++j)
#pragma unroll
                            for (int s = 0; s < D / 64; ++s)
                                tma_store_4d(kv == 0 ? &mapK : &mapV, sbase + L::kOut + j * (kTileRows * D * 2) + s * (kTileRows * 128),
                                             s * 64, hk0 + j, t0, b);
                        tma_store_commit();
                    }
                }
            }
            // this warp has read its lanes of the set: one arrival per warp on the even CTA's barrier
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];"
                             ::"r"(cluster_map_shared(bar_acc_empty(set), 0)) : "memory");
        }
        if (tid == 64) tma_store_wait_all();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag != 0 && tid == 0) {
        const uint64_t t_start = globaltimer_ns();
        while (globaltimer_ns() - t_start < 2000000ull) {}     // abort path only: let copies in flight land
    }
    // neither CTA leaves (or frees tensor memory) while the other may still read its accumulator or have loads in flight
    cluster_sync_all();
    if (warp == 1) tmem_dealloc_pair(tmem, kTmemCols);
}

}  // namespace moda
