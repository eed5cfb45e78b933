// MoDA forward kernel, wide variant: two softmax warpgroups and (for d = 64) three score buffers.
// Same operator, boundary and data layout as moda_fwd_kernel (see moda_fwd.cuh); used where the
// exponentials, not the tensor pipe, set the pace (d = 64: a 128x128 score tile costs 1024 SFU cycles
// but only 512 tensor cycles), and where TMEM has room for a third score buffer (O and o_d take
// 64 columns each at d = 64).
//
// One CTA owns one (b, h, 128-query-row tile).  512 threads, four warpgroups:
//
//   warps 0-3, 4-7   softmax A / B: one thread per query row in each.  The two warpgroups take
//                    alternate 128-key tiles (A: even j, B: odd j); with three score buffers the
//                    next tile of each is already computed when it finishes one, so the
//                    exponentials of one tile overlap the load / max / store phases of the other and
//                    keep the SFU pipe busy.  A thread reads S_j from TMEM, writes
//                    P_j = exp2(S_j c - m) as packed bf16 back over S_j's columns and keeps a partial
//                    row sum.  Both warpgroups share one reference maximum per row (shared memory,
//                    published right after the max phase of each tile); the O accumulator in TMEM is
//                    rescaled only when that reference grows by more than 2^8.  Both run the
//                    epilogue (half of the feature columns each).
//   warps 8-11       depth: as in moda_fwd_kernel (bulk-copy ring, partial softmax state, o_d in TMEM).
//   warp 12          TMA producer: Q tile, then K_j / V_j tiles (128B swizzle), one stage per score buffer.
//   warp 13          MMA issuer for S_j = Q K_j^T; owns TMEM.
//   warp 14          depth-cache producer (bulk copies).
//   warp 15          MMA issuer for O += P_j V_j.
//
// TMEM columns (fp32): S/P buffer b = j mod stages at [128 b, 128 b + 128); then O (D columns) and
// o_d (D columns): d = 64: 3 buffers, O at 384, o_d at 448 (d = 128 would get 2 buffers, O at 256,
// o_d at 384).
#pragma once

#include "moda_cache.cuh"
#include "moda_fwd.cuh"
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kFwd2Threads = 512;
constexpr int kMaxDynamicSmem = 232448;     // 227 KiB: the most one CTA can have on sm_100
constexpr int kFwdBN = 128;                 // keys per inner tile

template <int D, bool FP8 = false>
struct Fwd2Smem {
    static constexpr int kTileBytes = kTileRows * D * 2;          // one 128 x D bf16 tile
    static constexpr int kSubBytes = kTileRows * 128;             // one 128 x 64 sub-tile
    // K / V ring stages = score buffers in TMEM.  d = 64 leaves TMEM room for a third buffer, which
    // is what lets the two softmax warpgroups run without waiting for each other's P to be consumed.
    static constexpr int kStages = (D == 64) ? 3 : 2;
    static constexpr int kKeyTileBytes = kFwdBN * D * 2;          // one BN x D bf16 key / value tile
    static constexpr int kKeySubBytes = kFwdBN * 128;             // one BN x 64 sub-tile
    static constexpr int kQ = 0;
    static constexpr int kK = kQ + kTileBytes;                    // kStages stages
    static constexpr int kV = kK + kStages * kKeyTileBytes;       // kStages stages
    static constexpr int kU = kV + kStages * kKeyTileBytes;       // depth scores [32][128] fp32
    static constexpr int kMd = kU + 32 * kTileRows * 4;           // m_d [128], l_d [128]
    static constexpr int kMref = kMd + 2 * kTileRows * 4;         // shared reference maximum [128]
    static constexpr int kLx = kMref + kTileRows * 4;             // partial row sums of warpgroup B [128]
    static constexpr int kRing = kLx + kTileRows * 4;             // depth units: 8 chunks x 128 rows x 16 B
    // bf16 cache: 16 KiB units (8 feature chunks of one slot); e4m3 cache: all d features of one slot (128 d bytes)
    // with the 128 row scales beside them (moda_cache.cuh)
    static constexpr int kUnitBytes = FP8 ? kTileRows * D : 8 * kTileRows * 16;
    static constexpr int kScaleBytes = FP8 ? kTileRows * 4 : 0;
    static constexpr int kRingStages = (D == 128) ? 3 : 5;
    static constexpr int kScale = kRing + kRingStages * kUnitBytes;   // [ring stage][128] fp32 (e4m3 only)
    static constexpr int kBars = kScale + kRingStages * kScaleBytes;
    static constexpr int kNumBars = 48;
    static constexpr int kMisc = kBars + kNumBars * 8;            // tmem base, abort flag
    static constexpr int kTotal = kMisc + 16;
    // Tiles must sit on 1024-byte boundaries (128B swizzle).  The dynamic segment is requested
    // 1024-aligned; the slack covers a base that is not, and the kernel checks that it fits.
    static constexpr int kDynamic = (kTotal + 1024 <= kMaxDynamicSmem) ? kTotal + 1024 : kMaxDynamicSmem;
    static_assert(kTotal <= kMaxDynamicSmem, "shared-memory plan does not fit");
};

enum Fwd2Bar : int {
    k2BarQ = 0,
    k2BarKFull = 1,    // +stage (4)
    k2BarVFull = 9,    // +stage (4)
    k2BarVEmpty = 13,  // +stage (4): PV_j complete (also what the lazy rescale waits on)
    k2BarSFull = 17,   // +buffer (4): S_j complete; also frees the K stage of tile j
    k2BarPFull = 21,   // +buffer (4)
    k2BarDepth = 25,
    k2BarOFinal = 26,  // single phase: every MMA of the CTA has completed
    k2BarDrain = 27,
    k2BarRef = 28,     // +(j & 1): the reference maximum for tile j has been published
    k2BarDFull = 30,   // +ring stage (<= 6): depth unit landed
    k2BarDEmpty = 36,  // +ring stage (<= 6): all 128 depth threads have read the unit
};




template <int D, bool FP8 = false>
__global__ void __launch_bounds__(kFwd2Threads, 1)
moda_fwd2_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
                const FwdParams p) {
    using L = Fwd2Smem<D, FP8>;
    constexpr int NSUB = D / 64;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColO = L::kStages * 128, kColOd = kColO + ((D == 128) ? 128 : 64);

    if (g_moda_status != 0) return;   // an earlier kernel gave up a wait: do not pile up more timeouts

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = aligned_dynamic_smem(smem_raw, L::kTotal);
    if (smem == nullptr) {
        if (threadIdx.x == 0) atomicCAS(&g_moda_status, 0, kStatusSmemLayout);
        return;
    }
    const uint32_t sbase = smem_u32(smem);
    float* sU = reinterpret_cast<float*>(smem + L::kU);
    float* sMd = reinterpret_cast<float*>(smem + L::kMd);
    float* sLd = sMd + kTileRows;
    float* sMref = reinterpret_cast<float*>(smem + L::kMref);
    float* sLx = reinterpret_cast<float*>(smem + L::kLx);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar = [&](int i) { return sbase + L::kBars + 8u * uint32_t(i); };

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    const int nq = num_tiles(p.T);
    const TileCoord tc = tile_coord(blockIdx.x, nq, p.H, p.G);
    const int b = tc.b, h = tc.h, hk = tc.hk, qt = tc.qt;
    const int Hk = p.H / p.G;
    const int q0 = qt * kTileRows;
    // key tiles up to the one that holds the last row's own position (row i sees keys <= i + kv_off)
    const int n_kv = min((q0 + kTileRows + p.kv_off + kFwdBN - 1) / kFwdBN, (p.T_kv + kFwdBN - 1) / kFwdBN);

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(k2BarQ), 1);
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar(k2BarKFull + s), 1);
            mbar_init(bar(k2BarVFull + s), 1);
            mbar_init(bar(k2BarVEmpty + s), 1);
            mbar_init(bar(k2BarSFull + s), 1);
            mbar_init(bar(k2BarPFull + s), 128);
        }
        mbar_init(bar(k2BarRef + 0), 128);
        mbar_init(bar(k2BarRef + 1), 128);
        mbar_init(bar(k2BarDepth), 128);
        mbar_init(bar(k2BarOFinal), 1);
        mbar_init(bar(k2BarDrain), 1);
        for (int s = 0; s < L::kRingStages; ++s) {
            mbar_init(bar(k2BarDFull + s), 1);
            mbar_init(bar(k2BarDEmpty + s), 128);
        }
        fence_mbar_init();
    }
    if (warp == 13) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Register budget: the launch gives every warp 128 registers (4 warps per scheduler); the
    // producer warpgroup hands most of its share to the two softmax warpgroups.
    if (warp < 8) {
        // =========================== softmax A / B + epilogue ===========================
        setmaxnreg_inc<176>(); //SM
        const int wg = warp >> 2;                        // 0: even key tiles, 1: odd key tiles
        const int r = tid & 127;                         // query row inside the tile = TMEM lane
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        float my_ref = -INFINITY;                        // reference maximum (log2 domain) l_part is expressed in
        float l_part = 0.f;                              // this warpgroup's share of the row sum
        for (int j = wg; j < n_kv; j += 2) {
            const int buf = j % L::kStages;
            const uint32_t par = (j / L::kStages) & 1;
            const uint32_t tS = tmem + lane_addr + uint32_t(buf) * kFwdBN;
            mbar_wait(bar(k2BarSFull + buf), par, abort_flag, 10);
            tc_fence_after_sync();
            constexpr int NB = kFwdBN / 32;              // 32-column register blocks
            uint32_t sv[NB][32];
#pragma unroll
            for (int c = 0; c < NB; ++c) tmem_ld32(tS + c * 32, sv[c]);
            tmem_wait_ld();
            const int koff = j * kFwdBN - q0 - p.kv_off; // key of column c is visible to row r iff koff + c <= r
            if (koff + kFwdBN - 1 > 0) {                 // tiles that touch the diagonal: causal mask
#pragma unroll
                for (int c = 0; c < NB; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (koff + c * 32 + i > r) sv[c][i] = 0xff800000u;
            }
            float mx[NB];
#pragma unroll
            for (int c = 0; c < NB; ++c) {
                float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    m0 = max3(m0, __uint_as_float(sv[c][i]), __uint_as_float(sv[c][i + 1]));
                    m1 = max3(m1, __uint_as_float(sv[c][i + 2]), __uint_as_float(sv[c][i + 3]));
                }
                mx[c] = fmaxf(m0, m1);
            }
            float tile_max = mx[0];
#pragma unroll
            for (int c = 1; c < NB; ++c) tile_max = fmaxf(tile_max, mx[c]);
            tile_max *= p.scale_log2;
            // ---- agree on the reference maximum with the other warpgroup ----
            float m_prev = -INFINITY;
            if (j > 0) {
                mbar_wait(bar(k2BarRef + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag, 14);
                m_prev = sMref[r];
            }
            const float m_new = fmaxf(m_prev, tile_max);
            // j == 0: nothing accumulated yet, adopt the tile maximum.  Later: move the reference only
            // when some row of this warp grew by more than the threshold (decision per warp, because
            // the TMEM accesses of the rescale are warp-wide).
            const bool move = (j == 0) || __any_sync(0xffffffffu, m_new - m_prev > kRescaleThreshold);
            const float m_ref = move ? m_new : m_prev;
            sMref[r] = m_ref;
            mbar_arrive(bar(k2BarRef + (j & 1)));         // tile j+1 may now pick its reference
            if (move && j > 0) {
                // Bring O to the new reference.  O may only be touched between PV_{j-1} completing and
                // PV_j being issued; PV_j waits for this thread's arrival on k2BarPFull below.  PV_{j-1}
                // signals the V-stage barrier of tile j-1; its previous phase (PV_{j-5}) is known to be
                // complete because S_j was issued after PV_{j-4}.
                mbar_wait(bar(k2BarVEmpty + ((j - 1) % L::kStages)), ((j - 1) / L::kStages) & 1, abort_flag, 11);
                tc_fence_after_sync();
                const float f = fast_exp2(m_prev - m_ref);
#pragma unroll 1
                for (int c = 0; c < D / 16; ++c) {       // rare path: small chunks
                    uint32_t o[16];
                    tmem_ld16(tmem + lane_addr + kColO + c * 16, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st16(tmem + lane_addr + kColO + c * 16, o);
                }
            }
            if (my_ref != m_ref) {                       // re-express this warpgroup's partial sum
                l_part *= fast_exp2(my_ref - m_ref);     // (first tile: 0 * exp2(-inf) = 0)
                my_ref = m_ref;
            }
            const float neg_m = -m_ref;
            // P_j (bf16, two per column) overlays the first half of S_j's columns: one 32-column block of
            // scores at a time, stored as soon as it is converted.
            float sum0 = 0.f, sum1 = 0.f;
            auto exp_block = [&](const uint32_t (&sv)[32], uint32_t col) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    const float a0 = fast_exp2(fmaf(__uint_as_float(sv[2 * i]), p.scale_log2, neg_m));
                    const float a1 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 1]), p.scale_log2, neg_m));
                    const float b0 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 2]), p.scale_log2, neg_m));
                    const float b1 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 3]), p.scale_log2, neg_m));
                    sum0 += a0 + a1;
                    sum1 += b0 + b1;
                    pk[i] = pack_bf16x2(a0, a1);
                    pk[i + 1] = pack_bf16x2(b0, b1);
                }
                tmem_st16(tS + col, pk);
            };
#pragma unroll
            for (int c = 0; c < NB; ++c) exp_block(sv[c], c * 16);
            l_part += sum0 + sum1;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(k2BarPFull + buf));
        }

        // ------------------------------ epilogue ------------------------------
        // Final reference = the one published for the last tile; warpgroup B hands its partial sum
        // (in that reference) to A and vice versa through shared memory.
        mbar_wait(bar(k2BarRef + ((n_kv - 1) & 1)), ((n_kv - 1) >> 1) & 1, abort_flag, 15);
        const float m_seq = sMref[r];
        if (my_ref != m_seq) l_part = (my_ref == -INFINITY) ? 0.f : l_part * fast_exp2(my_ref - m_seq);
        if (wg == 1) sLx[r] = l_part;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        float l_seq = l_part;
        if (wg == 0) {                                   // row r of A is the only other user of sLx[r]
            l_seq += sLx[r];
            sLx[r] = l_seq;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (wg == 1) l_seq = sLx[r];

        mbar_wait(bar(k2BarOFinal), 0, abort_flag, 12);
        tc_fence_after_sync();
        float a_s = 1.f, a_d = 0.f, m_fin = m_seq, l_fin = l_seq;
        if (p.l > 0) {
            mbar_wait(bar(k2BarDepth), 0, abort_flag, 13);
            tc_fence_after_sync();
            const float m_d = sMd[r], l_d = sLd[r];
            m_fin = fmaxf(m_seq, m_d);
            a_s = fast_exp2(m_seq - m_fin);
            a_d = fast_exp2(m_d - m_fin);
            l_fin = a_s * l_seq + a_d * l_d;
        }
        const float inv = 1.f / l_fin;
        a_s *= inv;
        a_d *= inv;
        // O tile -> shared memory (the Q buffer, in the same swizzled layout) -> TMA store.
        // Warpgroup A converts the first half of the feature columns, B the second half.
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {
            const int c = wg * (D / 64) + cc;            // 32-column block index
            uint32_t o[32];
            tmem_ld32(tmem + lane_addr + kColO + c * 32, o);
            tmem_wait_ld();
            float of[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) of[i] = __uint_as_float(o[i]) * a_s;
            if (p.l > 0) {
                uint32_t od[32];
                tmem_ld32(tmem + lane_addr + kColOd + c * 32, od);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) of[i] = fmaf(__uint_as_float(od[i]), a_d, of[i]);
            }
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint4 v;
                v.x = pack_bf16x2(of[8 * g + 0], of[8 * g + 1]);
                v.y = pack_bf16x2(of[8 * g + 2], of[8 * g + 3]);
                v.z = pack_bf16x2(of[8 * g + 4], of[8 * g + 5]);
                v.w = pack_bf16x2(of[8 * g + 6], of[8 * g + 7]);
                *reinterpret_cast<uint4*>(smem + L::kQ + swz_chunk_offset(r, c * 4 + g)) = v;
            }
        }
        if (wg == 0 && q0 + r < p.T) p.LSE[(size_t(b) * p.H + h) * p.T + q0 + r] = (m_fin + log2f(l_fin)) * kLn2;
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0) {
#pragma unroll
            for (int s = 0; s < NSUB; ++s)
                tma_store_4d(&mapO, sbase + L::kQ + s * L::kSubBytes, s * 64, h, q0, b);
            tma_store_commit();
            tma_store_wait_all();
        }
    } else if (warp < 12) {
        // =========================== depth partial state ===========================
        setmaxnreg_dec<120>(); //DP
        if (p.l > 0) {
            const int r = tid - 256;
            const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
            mbar_wait(bar(k2BarQ), 0, abort_flag, 20);
            int unit = 0;                                 // running index into the producer's unit sequence
            // Reads this thread's 8 x 16 bytes of the next depth unit from the ring and frees the stage.
            auto take_unit = [&](uint4 (&dst)[8]) {
                const int st = unit % L::kRingStages;
                mbar_wait(bar(k2BarDFull + st), (unit / L::kRingStages) & 1, abort_flag, 21);
                const uint8_t* src = smem + L::kRing + st * L::kUnitBytes + r * 16;
#pragma unroll
                for (int c = 0; c < 8; ++c) dst[c] = *reinterpret_cast<const uint4*>(src + c * (kTileRows * 16));
                // The stage is refilled by the async proxy (bulk copy) while these loads went through the
                // generic proxy: the proxy fence orders them before the refill that this arrival allows.
                fence_proxy_async_smem();
                mbar_arrive(bar(k2BarDEmpty + st));
                ++unit;
            };
            // The slots are handled in groups of kFwdDepthGroup (the score scratch holds one group): an
            // online softmax over the groups, with the partial output o_d rescaled in TMEM when a later
            // group raises the maximum.  Up to 32 slots are one group.
            float m_d = -INFINITY, l_d = 0.f;
            if constexpr (FP8) {
                // e4m3 cache (see moda_fwd_kernel): a unit = all D features of one slot for the tile's rows + row scales
                constexpr int C8 = D / 16;
                const float* sScale = reinterpret_cast<const float*>(smem + L::kScale);
                auto take_unit8 = [&](uint4 (&dst)[C8], float& sc) {
                    const int st = unit % L::kRingStages;
                    mbar_wait(bar(k2BarDFull + st), (unit / L::kRingStages) & 1, abort_flag, 21);
                    const uint8_t* src = smem + L::kRing + st * L::kUnitBytes + r * 16;
#pragma unroll
                    for (int c = 0; c < C8; ++c) dst[c] = *reinterpret_cast<const uint4*>(src + c * (kTileRows * 16));
                    sc = sScale[st * kTileRows + r];
                    fence_proxy_async_smem();
                    mbar_arrive(bar(k2BarDEmpty + st));
                    ++unit;
                };
#pragma unroll 1
                for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                    const int gl = min(kFwdDepthGroup, p.l - g0);
                    {
                        float q[D];
#pragma unroll
                        for (int c = 0; c < D / 8; ++c) {
                            const uint4 v = *reinterpret_cast<const uint4*>(smem + L::kQ + swz_chunk_offset(r, c));
                            q[8 * c + 0] = bf16_lo_to_f32(v.x); q[8 * c + 1] = bf16_hi_to_f32(v.x);
                            q[8 * c + 2] = bf16_lo_to_f32(v.y); q[8 * c + 3] = bf16_hi_to_f32(v.y);
                            q[8 * c + 4] = bf16_lo_to_f32(v.z); q[8 * c + 5] = bf16_hi_to_f32(v.z);
                            q[8 * c + 6] = bf16_lo_to_f32(v.w); q[8 * c + 7] = bf16_hi_to_f32(v.w);
                        }
#pragma unroll 1
                        for (int i = 0; i < gl; ++i) {
                            uint4 cur[C8];
                            float sc;
                            take_unit8(cur, sc);
                            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                            for (int c = 0; c < C8; ++c) {
                                const uint32_t w[4] = {cur[c].x, cur[c].y, cur[c].z, cur[c].w};
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    float f0, f1, f2, f3;
                                    e4m3x4_to_f32(w[k], f0, f1, f2, f3);
                                    a0 = fmaf(q[16 * c + 4 * k + 0], f0, a0);
                                    a1 = fmaf(q[16 * c + 4 * k + 1], f1, a1);
                                    a2 = fmaf(q[16 * c + 4 * k + 2], f2, a2);
                                    a3 = fmaf(q[16 * c + 4 * k + 3], f3, a3);
                                }
                            }
                            sU[i * kTileRows + r] = ((a0 + a1) + (a2 + a3)) * sc;
                        }
                    }
                    float m_new = m_d;
                    for (int i = 0; i < gl; ++i) m_new = fmaxf(m_new, sU[i * kTileRows + r] * p.scale_log2);
                    const float f = fast_exp2(m_d - m_new);
                    l_d *= f;
                    for (int i = 0; i < gl; ++i) {
                        const float w = fast_exp2(fmaf(sU[i * kTileRows + r], p.scale_log2, -m_new));
                        sU[i * kTileRows + r] = w;
                        l_d += w;
                    }
                    m_d = m_new;
                    {
                        float acc[D];
                        if (g0 == 0) {
#pragma unroll
                            for (int c = 0; c < D; ++c) acc[c] = 0.f;
                        } else {
#pragma unroll
                            for (int c = 0; c < D / 32; ++c) {
                                uint32_t o[32];
                                tmem_ld32(tmem + lane_addr + kColOd + c * 32, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) acc[32 * c + i] = __uint_as_float(o[i]) * f;
                            }
                        }
#pragma unroll 1
                        for (int i = 0; i < gl; ++i) {
                            uint4 cur[C8];
                            float sc;
                            take_unit8(cur, sc);
                            const float w = sU[i * kTileRows + r] * sc;
#pragma unroll
                            for (int c = 0; c < C8; ++c) {
                                const uint32_t ww[4] = {cur[c].x, cur[c].y, cur[c].z, cur[c].w};
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    float f0, f1, f2, f3;
                                    e4m3x4_to_f32(ww[k], f0, f1, f2, f3);
                                    acc[16 * c + 4 * k + 0] = fmaf(w, f0, acc[16 * c + 4 * k + 0]);
                                    acc[16 * c + 4 * k + 1] = fmaf(w, f1, acc[16 * c + 4 * k + 1]);
                                    acc[16 * c + 4 * k + 2] = fmaf(w, f2, acc[16 * c + 4 * k + 2]);
                                    acc[16 * c + 4 * k + 3] = fmaf(w, f3, acc[16 * c + 4 * k + 3]);
                                }
                            }
                        }
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t o[32];
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(acc[32 * c + i]);
                            tmem_st32(tmem + lane_addr + kColOd + c * 32, o);
                        }
                        tmem_wait_st();
                    }
                }
            } else {
#pragma unroll 1
            for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                const int gl = min(kFwdDepthGroup, p.l - g0);
                // ---- depth scores u_i = <q, kd_i>, 64 features per sweep ----
#pragma unroll 1
                for (int half = 0; half < NSUB; ++half) {
                    float q[64];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 v = *reinterpret_cast<const uint4*>(smem + L::kQ + swz_chunk_offset(r, half * 8 + c));
                        q[8 * c + 0] = bf16_lo_to_f32(v.x); q[8 * c + 1] = bf16_hi_to_f32(v.x);
                        q[8 * c + 2] = bf16_lo_to_f32(v.y); q[8 * c + 3] = bf16_hi_to_f32(v.y);
                        q[8 * c + 4] = bf16_lo_to_f32(v.z); q[8 * c + 5] = bf16_hi_to_f32(v.z);
                        q[8 * c + 6] = bf16_lo_to_f32(v.w); q[8 * c + 7] = bf16_hi_to_f32(v.w);
                    }
#pragma unroll 1
                    for (int i = 0; i < gl; ++i) {
                        uint4 cur[8];
                        take_unit(cur);
                        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            a0 = fmaf(q[8 * c + 0], bf16_lo_to_f32(cur[c].x), a0);
                            a1 = fmaf(q[8 * c + 1], bf16_hi_to_f32(cur[c].x), a1);
                            a2 = fmaf(q[8 * c + 2], bf16_lo_to_f32(cur[c].y), a2);
                            a3 = fmaf(q[8 * c + 3], bf16_hi_to_f32(cur[c].y), a3);
                            a0 = fmaf(q[8 * c + 4], bf16_lo_to_f32(cur[c].z), a0);
                            a1 = fmaf(q[8 * c + 5], bf16_hi_to_f32(cur[c].z), a1);
                            a2 = fmaf(q[8 * c + 6], bf16_lo_to_f32(cur[c].w), a2);
                            a3 = fmaf(q[8 * c + 7], bf16_hi_to_f32(cur[c].w), a3);
                        }
                        const float part = (a0 + a1) + (a2 + a3);
                        if (half == 0) sU[i * kTileRows + r] = part;
                        else sU[i * kTileRows + r] += part;
                    }
                }
                // ---- partial softmax over the depth scores seen so far ----
                float m_new = m_d;
                for (int i = 0; i < gl; ++i) m_new = fmaxf(m_new, sU[i * kTileRows + r] * p.scale_log2);
                const float f = fast_exp2(m_d - m_new);       // first group: exp2(-inf) = 0
                l_d *= f;
                for (int i = 0; i < gl; ++i) {
                    const float w = fast_exp2(fmaf(sU[i * kTileRows + r], p.scale_log2, -m_new));
                    sU[i * kTileRows + r] = w;
                    l_d += w;
                }
                m_d = m_new;
                // ---- o_d = sum_i w_i vd_i, 64 features per sweep, parked in TMEM ----
#pragma unroll 1
                for (int half = 0; half < NSUB; ++half) {
                    float acc[64];
                    if (g0 == 0) {
#pragma unroll
                        for (int c = 0; c < 64; ++c) acc[c] = 0.f;
                    } else {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tmem + lane_addr + kColOd + half * 64 + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[32 * c + i] = __uint_as_float(o[i]) * f;
                        }
                    }
#pragma unroll 1
                    for (int i = 0; i < gl; ++i) {
                        uint4 cur[8];
                        take_unit(cur);
                        const float w = sU[i * kTileRows + r];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            acc[8 * c + 0] = fmaf(w, bf16_lo_to_f32(cur[c].x), acc[8 * c + 0]);
                            acc[8 * c + 1] = fmaf(w, bf16_hi_to_f32(cur[c].x), acc[8 * c + 1]);
                            acc[8 * c + 2] = fmaf(w, bf16_lo_to_f32(cur[c].y), acc[8 * c + 2]);
                            acc[8 * c + 3] = fmaf(w, bf16_hi_to_f32(cur[c].y), acc[8 * c + 3]);
                            acc[8 * c + 4] = fmaf(w, bf16_lo_to_f32(cur[c].z), acc[8 * c + 4]);
                            acc[8 * c + 5] = fmaf(w, bf16_hi_to_f32(cur[c].z), acc[8 * c + 5]);
                            acc[8 * c + 6] = fmaf(w, bf16_lo_to_f32(cur[c].w), acc[8 * c + 6]);
                            acc[8 * c + 7] = fmaf(w, bf16_hi_to_f32(cur[c].w), acc[8 * c + 7]);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(acc[32 * c + i]);
                        tmem_st32(tmem + lane_addr + kColOd + half * 64 + c * 32, o);
                    }
                    tmem_wait_st();                          // a later group reads these columns back
                }
            }
            }
            sMd[r] = m_d;
            sLd[r] = l_d;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(k2BarDepth));
        }
        if (p.append_slot != nullptr && h == hk * p.G) {
            // the "write" step of the depth stream (see moda_fwd_kernel): after this CTA's reads of the depth cache
            append_rows_from_global<D, FP8>(p.append_slot, p.K, p.V, b, hk, p.H / p.G, p.T, nq, qt, tid - 256);
        }
    } else {
      setmaxnreg_dec<40>();   // one instruction for the whole producer warpgroup (warps 12-15)
      if (warp == 12) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            mbar_arrive_expect_tx(bar(k2BarQ), L::kTileBytes);
#pragma unroll
            for (int s = 0; s < NSUB; ++s)
                tma_load_4d(sbase + L::kQ + s * L::kSubBytes, &mapQ, bar(k2BarQ), s * 64, h, q0, b);
            for (int j = 0; j < n_kv; ++j) {
                const int st = j % L::kStages;
                const uint32_t par = ((j / L::kStages) - 1) & 1;
                if (j >= L::kStages) mbar_wait(bar(k2BarSFull + st), par, abort_flag, 30);   // S of the stage's last tile is complete
                mbar_arrive_expect_tx(bar(k2BarKFull + st), L::kKeyTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s)
                    tma_load_4d(sbase + L::kK + st * L::kKeyTileBytes + s * L::kKeySubBytes, &mapK, bar(k2BarKFull + st),
                                s * 64, hk, j * kFwdBN, b);
                if (j >= L::kStages) mbar_wait(bar(k2BarVEmpty + st), par, abort_flag, 31);
                mbar_arrive_expect_tx(bar(k2BarVFull + st), L::kKeyTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s)
                    tma_load_4d(sbase + L::kV + st * L::kKeyTileBytes + s * L::kKeySubBytes, &mapV, bar(k2BarVFull + st),
                                s * 64, hk, j * kFwdBN, b);
            }
        }
      } else if (warp == 13) {
        // =========================== MMA issuer: S_j = Q K_j^T ===========================
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_s = make_idesc_bf16(128, kFwdBN, false, false);
            // every descriptor is built once; inside the loop a descriptor is one 64-bit add (the
            // start-address field counts 16-byte units and stays inside its 14 bits below 256 KiB)
            uint64_t dq[D / 16];
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) dq[kk] = desc_kmajor_sw128(sbase + L::kQ + (kk >> 2) * L::kSubBytes, kk & 3);
            const uint64_t dk0 = desc_kmajor_sw128(sbase + L::kK, 0);
            mbar_wait(bar(k2BarQ), 0, abort_flag, 41);
            for (int j = 0; j < n_kv; ++j) {
                const int st = j % L::kStages;
                // score buffer st still holds P_{j-stages} until that tile's PV has completed
                if (j >= L::kStages)
                    mbar_wait2(bar(k2BarKFull + st), (j / L::kStages) & 1, bar(k2BarVEmpty + st), ((j / L::kStages) - 1) & 1,
                               abort_flag, 40, 44);
                else
                    mbar_wait(bar(k2BarKFull + st), (j / L::kStages) & 1, abort_flag, 40);
                tc_fence_after_sync();
                const uint64_t dk = dk0 + uint64_t((st * L::kKeyTileBytes) >> 4);
                const uint32_t ts = tmem + uint32_t(st) * kFwdBN;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    umma_ss(ts, dq[kk], dk + uint64_t(((kk >> 2) * L::kKeySubBytes + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                umma_commit(bar(k2BarSFull + st));
            }
            if (*abort_flag != 0) {
                // A wait gave up somewhere: make sure no MMA of this warp is still in flight before TMEM is released.
                umma_commit(bar(k2BarDrain));
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar(k2BarDrain), 0) && globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
      } else if (warp == 15) {
        // =========================== MMA issuer: O += P_j V_j ===========================
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_o = make_idesc_bf16(128, D, false, true);
            const uint64_t dv0 = desc_mnmajor_sw128(sbase + L::kV, 0, L::kKeySubBytes);
            for (int j = 0; j < n_kv; ++j) {
                const int st = j % L::kStages;
                const uint32_t par = (j / L::kStages) & 1;
                mbar_wait2(bar(k2BarVFull + st), par, bar(k2BarPFull + st), par, abort_flag, 42, 43);
                tc_fence_after_sync();
                const uint64_t dv = dv0 + uint64_t((st * L::kKeyTileBytes) >> 4);
                const uint32_t tp = tmem + uint32_t(st) * kFwdBN;
                umma_ts(tmem + kColO, tp, dv, idesc_o, j > 0);
#pragma unroll
                for (int kk = 1; kk < kFwdBN / 16; ++kk)
                    umma_ts(tmem + kColO, tp + kk * 8, dv + uint64_t(kk * 128), idesc_o, 1);
                umma_commit(bar(k2BarVEmpty + st));
            }
            // All S MMAs completed before the P they fed was written, so the last PV is the last MMA.
            umma_commit(bar(k2BarOFinal));
            if (*abort_flag != 0) {
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar(k2BarOFinal), 0) && globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
      } else if (warp == 14) {
        // =========================== depth-cache producer ===========================
        // Streams the tile's depth keys, then values, as 16 KiB units (8 feature chunks of one slot:
        // one contiguous run of the cache) through the ring, in the order the depth warps consume
        // them.  The ring keeps up to kRingStages x 16 KiB of HBM reads in flight per SM.
        if (FP8 && lane == 0 && p.l > 0) {
            // e4m3 cache: one unit per (slot, K or V): the block's codes, and its 128 row scales behind them
            const uint64_t policy = l2_policy_evict_first();
            const size_t slot_bytes = cache8_slot_bytes(p.B, p.T, Hk, D);
            const size_t blk_bytes = cache8_block_bytes(D);
            const uint8_t* blk = reinterpret_cast<const uint8_t*>(p.depth_kv) + (((size_t(b) * Hk + hk) * nq + qt) * 2) * blk_bytes;
            int unit = 0;
            for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                const int gl = min(kFwdDepthGroup, p.l - g0);
                for (int kv = 0; kv < 2; ++kv)
                    for (int i = 0; i < gl; ++i, ++unit) {
                        const int st = unit % L::kRingStages;
                        if (unit >= L::kRingStages)
                            mbar_wait(bar(k2BarDEmpty + st), ((unit / L::kRingStages) - 1) & 1, abort_flag, 32);
                        mbar_arrive_expect_tx(bar(k2BarDFull + st), L::kUnitBytes + L::kScaleBytes);
                        const uint8_t* src = blk + size_t(g0 + i) * slot_bytes + size_t(kv) * blk_bytes;
                        bulk_load(sbase + L::kRing + st * L::kUnitBytes, src, L::kUnitBytes, bar(k2BarDFull + st), policy);
                        bulk_load(sbase + L::kScale + st * L::kScaleBytes, src + L::kUnitBytes, L::kScaleBytes, bar(k2BarDFull + st), policy);
                    }
            }
        } else if (lane == 0 && p.l > 0) {
            const uint64_t policy = l2_policy_evict_first();          // the depth cache is read exactly once
            const size_t slot_bytes = cache_slot_elems(p.B, p.T, Hk, D) * 2;
            const uint8_t* blk = reinterpret_cast<const uint8_t*>(p.depth_kv) +
                                 (((size_t(b) * Hk + hk) * nq + qt) * 2) * (size_t(kTileRows) * D * 2);
            int unit = 0;
            for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                const int gl = min(kFwdDepthGroup, p.l - g0);
                for (int kv = 0; kv < 2; ++kv)
                    for (int half = 0; half < NSUB; ++half)
                        for (int i = 0; i < gl; ++i, ++unit) {
                            const int st = unit % L::kRingStages;
                            if (unit >= L::kRingStages)
                                mbar_wait(bar(k2BarDEmpty + st), ((unit / L::kRingStages) - 1) & 1, abort_flag, 32);
                            mbar_arrive_expect_tx(bar(k2BarDFull + st), L::kUnitBytes);
                            bulk_load(sbase + L::kRing + st * L::kUnitBytes,
                                      blk + size_t(g0 + i) * slot_bytes + size_t(kv) * (size_t(kTileRows) * D * 2) + size_t(half) * L::kUnitBytes,
                                      L::kUnitBytes, bar(k2BarDFull + st), policy);
                        }
            }
        }
      }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag != 0 && tid == 256) {
        // Abort path only: give bulk copies still in flight a bounded time to land before the CTA's
        // shared memory is handed to another CTA.
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) {}
    }
    __syncthreads();
    if (warp == 13) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace moda
