// MoDA forward kernel for sm_100a (Sec. 2.2 definition; Alg. 1 gives the blockwise
// online-softmax schedule this kernel re-designs for tcgen05 / TMEM / TMA).
//
// One CTA owns one (b, query head h) and either one 128-query-row tile or, for causal calls over as many
// keys as queries, a pair of them (pair_coord: the p-th tile from the end, then the p-th from the start, so that
// every CTA has the same number of key tiles and the short tile's depth slots are worked on during the long
// tile's key loop); with grouped-query attention the G heads that share a key/value head are adjacent CTAs
// (tile_coord).  The rings and their phase counters run on across the two tiles.  384 threads, three warpgroups:
//
//   warps 0-3  softmax   one thread per query row.  Reads the score tile S_j from TMEM,
//                        keeps the running (m, l) of the online softmax in registers, writes
//                        P_j = exp2(S_j c - m) as packed bf16 back into the TMEM columns of
//                        S_j, rescales the O accumulator only when the running maximum grew
//                        by more than 2^8, and runs the epilogue (output tile, LSE).
//   warps 4-7  depth     one thread per query row (its q comes straight from global memory).  Reads the
//                        row's l depth keys/values (bf16, or e4m3 codes with row scales) from
//                        a shared-memory ring that warp 10 fills with 16 KiB bulk copies of
//                        the depth cache, builds an independent partial softmax state
//                        (m_d, l_d, o_d) on the CUDA cores (slots in groups of 32, online
//                        softmax over the groups) and parks o_d in TMEM.  Merging two partial
//                        softmax states is exact, so the epilogue obtains the single softmax
//                        over sequence and depth keys that the paper defines.  Afterwards it writes the
//                        layer's own K, V rows into a cache slot when the call asks for it.
//   warp 8     TMA       one lane streams the Q tile and the K_j / V_j tiles (128B swizzle)
//                        through two-stage rings.
//   warp 9     MMA (S)   issues S_j = Q K_j^T (operands in shared memory); owns the TMEM
//                        allocation.  The whole warp runs the loop, an elected lane issues.
//   warp 10    depth producer (one lane)
//   warp 11    MMA (PV)  issues O += P_j V_j (P_j from TMEM, V_j MN-major in shared memory).
//                        One tcgen05.mma costs its issuing warp 40-100 cycles, as much as a
//                        128x128x16 MMA executes, so the two contractions are issued by two
//                        warps on different schedulers and ordered by mbarriers.
//
// TMEM columns (fp32): [0,128) S_0/P_0   [128,256) S_1/P_1   [256,256+D) O   [384,384+D) o_d.
// The depth scores never touch the tensor cores and no score matrix is ever materialised.
#pragma once

#include "moda_cache.cuh"
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kFwdThreads = 384;   // three warpgroups: softmax, depth, {TMA, MMA, 2 idle warps}
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

// KST = stages of the K ring.  Two let K_{j+1} load while S_j is still being computed; one (the
// load starts when S_j completes and overlaps the softmax of tile j) leaves room for a deeper depth
// ring, for shapes whose depth stream outweighs the sequence work (the host picks, see launch_fwd).
// FP8: the depth cache holds e4m3 codes with a scale per row (moda_cache.cuh); a unit is then all d features of one
// slot's keys (or values) of the tile, and its 128 row scales travel beside it.
template <int D, int KST = 2, bool FP8 = false>
struct FwdSmem {
    static constexpr int kTileBytes = kTileRows * D * 2;          // one 128 x D bf16 tile
    static constexpr int kSubBytes = kTileRows * 128;             // one 128 x 64 sub-tile
    static constexpr int kKStages = KST;
    static constexpr int kQ = 0;
    static constexpr int kK = kQ + kTileBytes;                    // KST stages
    static constexpr int kV = kK + KST * kTileBytes;              // 2 stages
    static constexpr int kU = kV + 2 * kTileBytes;                // depth scores [32][128] fp32
    static constexpr int kMd = kU + 32 * kTileRows * 4;           // m_d [128], l_d [128]
    static constexpr int kRing = kMd + 2 * kTileRows * 4;         // depth units: 8 chunks x 128 rows x 16 B
    static constexpr int kUnitBytes = FP8 ? kTileRows * D : 8 * kTileRows * 16;   // 16 KiB (bf16, and e4m3 at d = 128), contiguous in the cache
    static constexpr int kScaleBytes = FP8 ? kTileRows * 4 : 0;   // row scales of a unit
    static constexpr int kNumBars = 32;
    static constexpr int kSmemLimit = 232448;                     // 227 KiB per CTA on sm_100
    // bf16: 1024 bytes of slack for aligning the segment by hand; e4m3: no slack (the scales need it), the segment
    // is declared 1024-aligned and checked at run time
    static constexpr int kSlack = FP8 ? 0 : 1024;
    static constexpr int kRingFit = (kSmemLimit - kSlack - kRing - kNumBars * 8 - 16) / (kUnitBytes + kScaleBytes);
    static constexpr int kRingStages = kRingFit < 6 ? kRingFit : 6;   // every unit that fits, at most 6
    static_assert(kRingStages >= 3, "depth ring too shallow");
    static constexpr int kScale = kRing + kRingStages * kUnitBytes;   // [ring stage][128] fp32 (e4m3 only)
    static constexpr int kBars = kScale + kRingStages * kScaleBytes;
    static constexpr int kMisc = kBars + kNumBars * 8;            // tmem base, abort flag
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + kSlack;
};

enum FwdBar : int {
    kBarQ = 0,
    kBarKFull = 1,    // +stage
    kBarVFull = 5,    // +stage
    kBarVEmpty = 7,   // +stage: PV_j complete (V stage and score buffer free; O may be rescaled)
    kBarSFull = 9,    // +buffer: S_j complete (also frees the K stage)
    kBarPFull = 11,   // +buffer
    kBarDrain2 = 13,  // abort path of the second issuer
    kBarDepth = 14,
    kBarOFinal = 15,  // single phase: every MMA of the CTA has completed
    kBarDrain = 16,
    kBarDFull = 17,   // +ring stage (<= 6): depth unit landed
    kBarDEmpty = 23,  // +ring stage (<= 6): all 128 depth threads have read the unit
    kBarTileDone = 29,  // one phase per query tile of the CTA: its epilogue (output stored) is complete
};

// Depth slots per group of the forward's online softmax over the depth keys (one group's scores fit
// the shared-memory scratch); more slots than this take several groups.
constexpr int kFwdDepthGroup = 32;

struct FwdParams {
    const __nv_bfloat16* Q;          // [B][T][H][d]: the depth warps read their rows straight from global memory
    const __nv_bfloat16* K;          // [B][T_kv][H/G][d]: the write step reads the rows of the CTA's own positions from here
    const __nv_bfloat16* V;
    const void* depth_kv;            // cache layout (bf16, or e4m3 codes + scales), >= l slots (unused when l == 0)
    __nv_bfloat16* O;
    float* LSE;
    int B, T, H, l;                  // T query positions, H query heads
    int T_kv, kv_off;                // sequence keys 0 .. T_kv - 1; query row i sits at key position i + kv_off (kv_off = T_kv - T)
    int G;                           // query heads per key/value head (1 = plain multi-head attention)
    int pair;                        // nonzero: a CTA takes a pair of query tiles (see pair_coord), else one tile, heaviest first
    float scale_log2;                // scale * log2(e)
    // "Write" step of the depth stream fused into the forward: when not null, the base of one cache slot
    // (H / G heads) into which every CTA copies the K and V rows of its own positions (append_rows_from_global).
    // Only with kv_off == 0; the first head of a group writes.
    void* append_slot;               // bf16 slot, or (e4m3 instantiations) a slot of codes + row scales
};

// Which (batch, query head, key/value head, query tile) a CTA works on.  The G query heads that
// share a key/value head (Sec. 3, group-aware depth KV: rows with the same base time reuse the same
// depth blocks) are adjacent CTAs, so they run together and the depth block and the K/V tiles they
// share cross HBM once and are served by L2 to the others; inside a key/value head the heaviest
// query tiles come first.
struct TileCoord {
    int b, h, hk, qt;
};
__device__ __forceinline__ TileCoord tile_coord(int block, int nq, int H, int G) {
    const int per_kv = nq * G;
    const int bhk = block / per_kv, rem = block % per_kv;
    const int Hk = H / G;
    TileCoord c;
    c.b = bhk / Hk;
    c.hk = bhk % Hk;
    c.h = c.hk * G + rem % G;
    c.qt = nq - 1 - rem / G;
    return c;
}
// The d = 128 kernel gives a CTA a *pair* of query tiles of one head, the p-th from the end and the p-th from the
// start (one tile when they coincide): under the causal mask every pair has the same number of key tiles, and the
// depth stream of the short tile is worked on while the long tile's key loop still runs.
__host__ __device__ inline int num_tile_pairs(int nq) { return (nq + 1) / 2; }
__device__ __forceinline__ TileCoord pair_coord(int block, int nq, int H, int G) {
    TileCoord c = tile_coord(block, num_tile_pairs(nq), H, G);
    c.qt = num_tile_pairs(nq) - 1 - c.qt;        // pair index p; its tiles are nq - 1 - p (first) and p
    return c;
}

// Shared-memory address of 16-byte chunk `c` (0..D/8-1) of row `r` inside a 128 x D tile that
// TMA wrote as D/64 sub-tiles of [128][64] with the 128-byte swizzle.
__device__ __forceinline__ uint32_t swz_chunk_offset(int r, int c) {
    return uint32_t(c >> 3) * uint32_t(kTileRows * 128) + uint32_t(r) * 128u + (uint32_t((c & 7) ^ (r & 7)) << 4);
}

// "Write" step of the depth stream inside the forward: one thread copies the K row and the V row of one of the CTA's own
// positions from the input tensors into block (b, hk, qt) of a slot: chunk c of row r goes to [c][r], so a warp writes 512
// contiguous bytes per chunk.  The rows are read from global memory (the key loop loads the same rows as its diagonal
// tile, so they come from L2 or cost one more read of 4 d bytes per position), which lets the depth warps do this as
// soon as they have finished reading the cache, off the path of the key loop and the epilogue.  Rows past T are written
// as zeros (e4m3: code 0, scale 1), which is what the cache wants in its tail rows.
// FP8: the slot is in the e4m3 layout (moda_cache.cuh) and the row is quantised exactly as depth_cache_quant_kernel does
// (row maximum / 448 as the scale, correctly rounded quotients, round to nearest even, saturating; a zero row has scale 1).
template <int D, bool FP8>
__device__ __forceinline__ void append_rows_from_global(void* slot, const __nv_bfloat16* K, const __nv_bfloat16* V,
                                                        int b, int hk, int Hk, int T, int nq, int qt, int r) {
    constexpr int CH = D / 8;
    const int t = qt * kTileRows + r;
    const bool valid = t < T;
    const size_t block_index = (size_t(b) * Hk + hk) * nq + qt;
    const size_t row = ((size_t(b) * T + (valid ? t : 0)) * Hk + hk) * CH;
#pragma unroll 1
    for (int kv = 0; kv < 2; ++kv) {
        const uint4* src = reinterpret_cast<const uint4*>(kv == 0 ? K : V) + row;
        uint4 x[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c) x[c] = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
        if constexpr (!FP8) {
            uint4* dst = reinterpret_cast<uint4*>(slot) + (block_index * 2 + kv) * (kTileRows * CH) + r;
#pragma unroll
            for (int c = 0; c < CH; ++c) dst[c * kTileRows] = x[c];
        } else {
            uint8_t* blk = static_cast<uint8_t*>(slot) + (block_index * 2 + kv) * cache8_block_bytes(D);
            float am = 0.f;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const uint32_t w[4] = {x[c].x, x[c].y, x[c].z, x[c].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) am = fmaxf(am, fmaxf(fabsf(bf16_lo_to_f32(w[k])), fabsf(bf16_hi_to_f32(w[k]))));
            }
            const float scale = am > 0.f ? __fdiv_rn(am, 448.f) : 1.f;
            const RowDivider dv = make_row_divider(scale);
            uint4* codes = reinterpret_cast<uint4*>(blk) + r;
#pragma unroll
            for (int g = 0; g < D / 16; ++g) {            // 16 features per chunk of codes = two 16-byte bf16 chunks
                uint32_t cw[4];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint32_t w[4] = {x[2 * g + half].x, x[2 * g + half].y, x[2 * g + half].z, x[2 * g + half].w};
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        uint16_t lo, hi;
                        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo)
                            : "f"(div_rn(bf16_hi_to_f32(w[2 * k]), dv)), "f"(div_rn(bf16_lo_to_f32(w[2 * k]), dv)));
                        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi)
                            : "f"(div_rn(bf16_hi_to_f32(w[2 * k + 1]), dv)), "f"(div_rn(bf16_lo_to_f32(w[2 * k + 1]), dv)));
                        cw[2 * half + k] = uint32_t(lo) | (uint32_t(hi) << 16);
                    }
                }
                codes[g * kTileRows] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            }
            reinterpret_cast<float*>(blk + size_t(kTileRows) * D)[r] = scale;
        }
    }
}

template <int D, int KST = 2, bool FP8 = false>
__global__ void __launch_bounds__(kFwdThreads, 1)
moda_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
                const FwdParams p) {
    using L = FwdSmem<D, KST, FP8>;
    constexpr int NSUB = D / 64;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColO = 256, kColOd = 384;

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
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
    auto bar = [&](int i) { return sbase + L::kBars + 8u * uint32_t(i); };

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    const int nq = num_tiles(p.T);
    const bool paired = p.pair != 0;
    const TileCoord tc = paired ? pair_coord(blockIdx.x, nq, p.H, p.G) : tile_coord(blockIdx.x, nq, p.H, p.G);
    const int b = tc.b, h = tc.h, hk = tc.hk;
    const int Hk = p.H / p.G;
    // the CTA's query tiles, the longer one first; every role walks them in this order
    const int n_tiles = (paired && nq - 1 - tc.qt != tc.qt) ? 2 : 1;
    auto tile_qt = [&](int t) { return (paired && t == 0) ? nq - 1 - tc.qt : tc.qt; };
    // causal: key tiles up to the one that holds the last row's own position (row i sees keys <= i + kv_off)
    auto tile_nkv = [&](int t) {
        return min((tile_qt(t) * kTileRows + kTileRows + p.kv_off + kTileRows - 1) / kTileRows, num_tiles(p.T_kv));
    };

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(kBarQ), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarVFull + s), 1);
            mbar_init(bar(kBarVEmpty + s), 1);
            mbar_init(bar(kBarSFull + s), 1);
            mbar_init(bar(kBarPFull + s), 128);
        }
        mbar_init(bar(kBarDepth), 128);
        mbar_init(bar(kBarTileDone), 1);
        mbar_init(bar(kBarOFinal), 1);
        mbar_init(bar(kBarDrain), 1);
        mbar_init(bar(kBarDrain2), 1);
        for (int s = 0; s < L::kRingStages; ++s) {
            mbar_init(bar(kBarDFull + s), 1);
            mbar_init(bar(kBarDEmpty + s), 128);
        }
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

    // Register budget: the launch gives every warp 168 registers (3 warps per scheduler);
    // the producer warpgroup hands most of its share to the two compute warpgroups.
    if (warp < 4) {
        // =========================== softmax + epilogue ===========================
        setmaxnreg_inc<216>();
        const int r = tid;                               // query row inside the tile = TMEM lane
        const uint32_t lane_addr = uint32_t(warp * 32) << 16;
        int jbase = 0;                                   // key tiles of the CTA's earlier query tiles: the rings run on
        for (int t = 0; t < n_tiles; ++t) {
        const int qt = tile_qt(t), q0 = qt * kTileRows, n_kv = tile_nkv(t);
        float m_ref = -INFINITY;                         // reference maximum (log2 domain) the stored P, O use
        float l_sum = 0.f;
        for (int j = 0; j < n_kv; ++j) {
            const int jj = jbase + j;
            const int buf = jj & 1;
            const uint32_t tS = tmem + lane_addr + uint32_t(buf) * 128u;
            mbar_wait(bar(kBarSFull + buf), (jj >> 1) & 1, abort_flag, 10);
            tc_fence_after_sync();
            uint32_t s0[32], s1[32], s2[32], s3[32];
            tmem_ld32(tS + 0, s0);
            tmem_ld32(tS + 32, s1);
            tmem_ld32(tS + 64, s2);
            tmem_ld32(tS + 96, s3);
            tmem_wait_ld();
            if ((j + 1) * kTileRows - 1 > q0 + p.kv_off) {   // tile reaches past the first row's position: causal mask
                const int rs = r + q0 + p.kv_off - j * kTileRows;   // column i of this tile is visible iff i <= rs
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (i > rs) s0[i] = 0xff800000u;
                    if (i + 32 > rs) s1[i] = 0xff800000u;
                    if (i + 64 > rs) s2[i] = 0xff800000u;
                    if (i + 96 > rs) s3[i] = 0xff800000u;
                }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {            // 3-input max: one instruction per two scores
                mx0 = max3(mx0, __uint_as_float(s0[i]), __uint_as_float(s0[i + 1]));
                mx1 = max3(mx1, __uint_as_float(s1[i]), __uint_as_float(s1[i + 1]));
                mx2 = max3(mx2, __uint_as_float(s2[i]), __uint_as_float(s2[i + 1]));
                mx3 = max3(mx3, __uint_as_float(s3[i]), __uint_as_float(s3[i + 1]));
            }
            const float m_new = fmaxf(m_ref, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2);
            if (j == 0) {
                m_ref = m_new;                           // nothing accumulated yet
            } else if (__any_sync(0xffffffffu, m_new - m_ref > kRescaleThreshold)) {
                // The maximum grew a lot: bring O and l to the new reference.  O may only be
                // touched between PV_{j-1} completing and PV_j being issued; PV_j waits for
                // this thread's arrival on kBarPFull below.
                mbar_wait(bar(kBarVEmpty + ((jj - 1) & 1)), ((jj - 1) >> 1) & 1, abort_flag, 11);
                tc_fence_after_sync();
                const float f = fast_exp2(m_ref - m_new);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tmem + lane_addr + kColO + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st32(tmem + lane_addr + kColO + c * 32, o);
                }
                l_sum *= f;
                m_ref = m_new;
            }
            const float neg_m = -m_ref;
            float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
            uint32_t pk0[16], pk1[16], pk2[16], pk3[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float a0 = fast_exp2(fmaf(__uint_as_float(s0[2 * i]), p.scale_log2, neg_m));
                const float a1 = fast_exp2(fmaf(__uint_as_float(s0[2 * i + 1]), p.scale_log2, neg_m));
                const float b0 = fast_exp2(fmaf(__uint_as_float(s1[2 * i]), p.scale_log2, neg_m));
                const float b1 = fast_exp2(fmaf(__uint_as_float(s1[2 * i + 1]), p.scale_log2, neg_m));
                const float c0 = fast_exp2(fmaf(__uint_as_float(s2[2 * i]), p.scale_log2, neg_m));
                const float c1 = fast_exp2(fmaf(__uint_as_float(s2[2 * i + 1]), p.scale_log2, neg_m));
                const float d0 = fast_exp2(fmaf(__uint_as_float(s3[2 * i]), p.scale_log2, neg_m));
                const float d1 = fast_exp2(fmaf(__uint_as_float(s3[2 * i + 1]), p.scale_log2, neg_m));
                sum0 += a0 + a1; sum1 += b0 + b1; sum2 += c0 + c1; sum3 += d0 + d1;
                pk0[i] = pack_bf16x2(a0, a1);
                pk1[i] = pack_bf16x2(b0, b1);
                pk2[i] = pack_bf16x2(c0, c1);
                pk3[i] = pack_bf16x2(d0, d1);
            }
            l_sum += (sum0 + sum1) + (sum2 + sum3);
            // P_j (bf16, two per column) overlays the first 64 columns of S_j.
            tmem_st16(tS + 0, pk0);
            tmem_st16(tS + 16, pk1);
            tmem_st16(tS + 32, pk2);
            tmem_st16(tS + 48, pk3);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(kBarPFull + buf));
        }

        // ------------------------------ epilogue ------------------------------
        mbar_wait(bar(kBarOFinal), t & 1, abort_flag, 12);
        tc_fence_after_sync();
        float a_s = 1.f, a_d = 0.f, m_fin = m_ref, l_fin = l_sum;
        if (p.l > 0) {
            mbar_wait(bar(kBarDepth), t & 1, abort_flag, 13);
            tc_fence_after_sync();
            const float m_d = sMd[r], l_d = sLd[r];
            m_fin = fmaxf(m_ref, m_d);
            a_s = fast_exp2(m_ref - m_fin);
            a_d = fast_exp2(m_d - m_fin);
            l_fin = a_s * l_sum + a_d * l_d;
        }
        const float inv = 1.f / l_fin;
        a_s *= inv;
        a_d *= inv;
        // O tile -> shared memory (the Q buffer, in the same swizzled layout) -> TMA store.
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
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
        if (q0 + r < p.T) p.LSE[(size_t(b) * p.H + h) * p.T + q0 + r] = (m_fin + log2f(l_fin)) * kLn2;
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 0) {
#pragma unroll
            for (int s = 0; s < NSUB; ++s)
                tma_store_4d(&mapO, sbase + L::kQ + s * L::kSubBytes, s * 64, h, q0, b);
            tma_store_commit();
            tma_store_wait_all();
        }
        // The tile is done: the Q buffer (output staging), O and the depth partial in tensor memory may be reused for the
        // CTA's next tile.
        tc_fence_before_sync();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 0) mbar_arrive(bar(kBarTileDone));
        jbase += n_kv;
        }
    } else if (warp < 8) {
        // =========================== depth partial state ===========================
        setmaxnreg_inc<216>();
        if (p.l > 0) {
            const int r = tid - 128;
            const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
            int unit = 0;                                 // running index into the producer's unit sequence (over all tiles)
            // Reads this thread's 8 x 16 bytes of the next depth unit from the ring and frees the stage.
            auto take_unit = [&](uint4 (&dst)[8]) {
                const int st = unit % L::kRingStages;
                mbar_wait(bar(kBarDFull + st), (unit / L::kRingStages) & 1, abort_flag, 21);
                const uint8_t* src = smem + L::kRing + st * L::kUnitBytes + r * 16;
#pragma unroll
                for (int c = 0; c < 8; ++c) dst[c] = *reinterpret_cast<const uint4*>(src + c * (kTileRows * 16));
                // The stage is refilled by the async proxy (bulk copy) while these loads went through the
                // generic proxy: the proxy fence orders them before the refill that this arrival allows.
                fence_proxy_async_smem();
                mbar_arrive(bar(kBarDEmpty + st));
                ++unit;
            };
            // The slots are handled in groups of kFwdDepthGroup (the score scratch holds one group): an
            // online softmax over the groups, with the partial output o_d rescaled in TMEM when a later
            // group raises the maximum.  Up to 32 slots are one group.
            for (int t = 0; t < n_tiles; ++t) {
            const int qt = tile_qt(t), q0 = qt * kTileRows;
            // this thread's query row (zeros past T, as the TMA-loaded tile has them)
            const bool qvalid = q0 + r < p.T;
            const uint4* qrow = reinterpret_cast<const uint4*>(p.Q + ((size_t(b) * p.T + (qvalid ? q0 + r : 0)) * p.H + h) * D);
            // The depth partial of the CTA's previous tile stays parked (tensor memory, sMd / sLd) until that tile's
            // epilogue has read it; this tile's slots are streamed and used meanwhile, only the first store waits.
            auto wait_previous_tile = [&]() { if (t > 0) mbar_wait(bar(kBarTileDone), (t - 1) & 1, abort_flag, 25); };
            float m_d = -INFINITY, l_d = 0.f;
            if constexpr (FP8) {
                // e4m3 cache: a unit holds all D features of one slot's keys (values) for the tile's rows, its row
                // scales sit beside it; codes are widened to fp32 in registers, everything else as below.
                constexpr int C8 = D / 16;                    // 16-byte chunks (16 codes) of a row
                const float* sScale = reinterpret_cast<const float*>(smem + L::kScale);
                auto take_unit8 = [&](uint4 (&dst)[C8], float& sc) {
                    const int st = unit % L::kRingStages;
                    mbar_wait(bar(kBarDFull + st), (unit / L::kRingStages) & 1, abort_flag, 21);
                    const uint8_t* src = smem + L::kRing + st * L::kUnitBytes + r * 16;
#pragma unroll
                    for (int c = 0; c < C8; ++c) dst[c] = *reinterpret_cast<const uint4*>(src + c * (kTileRows * 16));
                    sc = sScale[st * kTileRows + r];
                    fence_proxy_async_smem();
                    mbar_arrive(bar(kBarDEmpty + st));
                    ++unit;
                };
#pragma unroll 1
                for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                    const int gl = min(kFwdDepthGroup, p.l - g0);
                    {   // ---- depth scores u_i = s_i <q, codes_i> ----
                        float q[D];
#pragma unroll
                        for (int c = 0; c < D / 8; ++c) {
                            const uint4 v = qvalid ? __ldg(qrow + c) : make_uint4(0u, 0u, 0u, 0u);
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
                    const float f = fast_exp2(m_d - m_new);       // first group: exp2(-inf) = 0
                    l_d *= f;
                    for (int i = 0; i < gl; ++i) {
                        const float w = fast_exp2(fmaf(sU[i * kTileRows + r], p.scale_log2, -m_new));
                        sU[i * kTileRows + r] = w;
                        l_d += w;
                    }
                    m_d = m_new;
                    {   // ---- o_d = sum_i (w_i s_i) codes_i, parked in TMEM ----
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
                        if (g0 == 0) wait_previous_tile();
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t o[32];
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(acc[32 * c + i]);
                            tmem_st32(tmem + lane_addr + kColOd + c * 32, o);
                        }
                        tmem_wait_st();                          // a later group reads these columns back
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
                        const uint4 v = qvalid ? __ldg(qrow + half * 8 + c) : make_uint4(0u, 0u, 0u, 0u);
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
                    if (g0 == 0 && half == 0) wait_previous_tile();
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
            mbar_arrive(bar(kBarDepth));
            }
        }
        if (p.append_slot != nullptr && h == hk * p.G) {
            // the write step: every read of the depth cache by this CTA is complete here, so the slot may be one that was read
            for (int t = 0; t < n_tiles; ++t)
                append_rows_from_global<D, FP8>(p.append_slot, p.K, p.V, b, hk, Hk, p.T, nq, tile_qt(t), tid - 128);
        }
    } else {
      setmaxnreg_dec<72>();   // one instruction for the whole producer warpgroup (warps 8-11)
      if (warp == 8) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            int jbase = 0;
            for (int t = 0; t < n_tiles; ++t) {
                const int q0 = tile_qt(t) * kTileRows, n_kv = tile_nkv(t);
                // the Q buffer doubles as the output staging of the previous tile
                if (t > 0) mbar_wait(bar(kBarTileDone), (t - 1) & 1, abort_flag, 33);
                mbar_arrive_expect_tx(bar(kBarQ), L::kTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s)
                    tma_load_4d(sbase + L::kQ + s * L::kSubBytes, &mapQ, bar(kBarQ), s * 64, h, q0, b);
                for (int j = 0; j < n_kv; ++j) {
                    const int jj = jbase + j;
                    const int st = jj & 1, kst = jj % KST;
                    // the K stage is free once S of its previous tile (jj - KST) has completed
                    if (jj >= KST) mbar_wait(bar(kBarSFull + ((jj - KST) & 1)), ((jj - KST) >> 1) & 1, abort_flag, 30);
                    mbar_arrive_expect_tx(bar(kBarKFull + kst), L::kTileBytes);
#pragma unroll
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_4d(sbase + L::kK + kst * L::kTileBytes + s * L::kSubBytes, &mapK, bar(kBarKFull + kst),
                                    s * 64, hk, j * kTileRows, b);
                    if (jj >= 2) mbar_wait(bar(kBarVEmpty + st), ((jj - 2) >> 1) & 1, abort_flag, 31);
                    mbar_arrive_expect_tx(bar(kBarVFull + st), L::kTileBytes);
#pragma unroll
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_4d(sbase + L::kV + st * L::kTileBytes + s * L::kSubBytes, &mapV, bar(kBarVFull + st),
                                    s * 64, hk, j * kTileRows, b);
                }
                jbase += n_kv;
            }
        }
      } else if (warp == 9) {
        // =========================== MMA issuer: S_j = Q K_j^T ===========================
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
            // every descriptor is built once; inside the loop a descriptor is one 64-bit add (the
            // start-address field counts 16-byte units and stays inside its 14 bits below 256 KiB)
            uint64_t dq[D / 16];
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) dq[kk] = desc_kmajor_sw128(sbase + L::kQ + (kk >> 2) * L::kSubBytes, kk & 3);
            const uint64_t dk0 = desc_kmajor_sw128(sbase + L::kK, 0);
            int jbase = 0;
            for (int t = 0; t < n_tiles; ++t) {
            const int n_kv = tile_nkv(t);
            mbar_wait(bar(kBarQ), t & 1, abort_flag, 41);
            for (int j = 0; j < n_kv; ++j) {
                const int jj = jbase + j;
                const int st = jj & 1, kst = jj % KST;
                // score buffer st still holds P_{jj-2} until PV_{jj-2} has completed
                if (jj >= 2) mbar_wait2(bar(kBarKFull + kst), (jj / KST) & 1, bar(kBarVEmpty + st), ((jj - 2) >> 1) & 1, abort_flag, 40, 44);
                else mbar_wait(bar(kBarKFull + kst), (jj / KST) & 1, abort_flag, 40);
                tc_fence_after_sync();
                const uint64_t dk = dk0 + uint64_t((kst * L::kTileBytes) >> 4);
                const uint32_t ts = tmem + uint32_t(st) * 128u;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    umma_ss(ts, dq[kk], dk + uint64_t(((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                umma_commit(bar(kBarSFull + st));
            }
            jbase += n_kv;
            }
            if (*abort_flag != 0) {
                // A wait gave up somewhere: make sure no MMA of this thread is still in flight before TMEM is released.
                umma_commit(bar(kBarDrain));
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar(kBarDrain), 0) && globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
      } else if (warp == 11) {
        // =========================== MMA issuer: O += P_j V_j ===========================
        {   // whole warp: operands are warp-uniform, one elected lane issues
            constexpr uint32_t idesc_o = make_idesc_bf16(128, D, false, true);
            const uint64_t dv0 = desc_mnmajor_sw128(sbase + L::kV, 0, L::kSubBytes);
            int jbase = 0;
            for (int t = 0; t < n_tiles; ++t) {
            const int n_kv = tile_nkv(t);
            for (int j = 0; j < n_kv; ++j) {
                const int jj = jbase + j;
                const int st = jj & 1;
                mbar_wait2(bar(kBarVFull + st), (jj >> 1) & 1, bar(kBarPFull + st), (jj >> 1) & 1, abort_flag, 42, 43);
                tc_fence_after_sync();
                const uint64_t dv = dv0 + uint64_t((st * L::kTileBytes) >> 4);
                const uint32_t tp = tmem + uint32_t(st) * 128u;
                umma_ts(tmem + kColO, tp, dv, idesc_o, j > 0);
#pragma unroll
                for (int kk = 1; kk < kTileRows / 16; ++kk)
                    umma_ts(tmem + kColO, tp + kk * 8, dv + uint64_t(kk * 128), idesc_o, 1);
                umma_commit(bar(kBarVEmpty + st));
            }
            // All S MMAs of the tile completed before the P they fed was written, so its last PV is its last MMA.
            umma_commit(bar(kBarOFinal));
            jbase += n_kv;
            }
            if (*abort_flag != 0) {
                // A wait gave up somewhere: make sure no MMA is still in flight before TMEM is released.
                umma_commit(bar(kBarDrain2));
                const uint64_t t0 = globaltimer_ns();
                while (!mbar_try_wait(bar(kBarDrain2), 0) && globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
      } else if (warp == 10) {
        // =========================== depth-cache producer ===========================
        // Streams the tile's depth keys, then values, as 16 KiB units (8 feature chunks of one slot:
        // one contiguous run of the cache) through the ring, in the order the depth warps consume
        // them.  The ring keeps up to kRingStages x 16 KiB of HBM reads in flight per SM.
        if (FP8 && lane == 0 && p.l > 0) {
            // e4m3 cache: one unit per (slot, K or V): the block's codes, and its 128 row scales behind them
            const uint64_t policy = l2_policy_evict_first();
            const size_t slot_bytes = cache8_slot_bytes(p.B, p.T, Hk, D);
            const size_t blk_bytes = cache8_block_bytes(D);
            int unit = 0;
            for (int t = 0; t < n_tiles; ++t) {
            const uint8_t* blk = reinterpret_cast<const uint8_t*>(p.depth_kv) + (((size_t(b) * Hk + hk) * nq + tile_qt(t)) * 2) * blk_bytes;
            for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                const int gl = min(kFwdDepthGroup, p.l - g0);
                for (int kv = 0; kv < 2; ++kv)
                    for (int i = 0; i < gl; ++i, ++unit) {
                        const int st = unit % L::kRingStages;
                        if (unit >= L::kRingStages)
                            mbar_wait(bar(kBarDEmpty + st), ((unit / L::kRingStages) - 1) & 1, abort_flag, 32);
                        mbar_arrive_expect_tx(bar(kBarDFull + st), L::kUnitBytes + L::kScaleBytes);
                        const uint8_t* src = blk + size_t(g0 + i) * slot_bytes + size_t(kv) * blk_bytes;
                        bulk_load(sbase + L::kRing + st * L::kUnitBytes, src, L::kUnitBytes, bar(kBarDFull + st), policy);
                        bulk_load(sbase + L::kScale + st * L::kScaleBytes, src + L::kUnitBytes, L::kScaleBytes, bar(kBarDFull + st), policy);
                    }
            }
            }
        } else if (lane == 0 && p.l > 0) {
            const uint64_t policy = l2_policy_evict_first();          // the depth cache is read exactly once
            const size_t slot_bytes = cache_slot_elems(p.B, p.T, Hk, D) * 2;
            int unit = 0;
            for (int t = 0; t < n_tiles; ++t) {
            const uint8_t* blk = reinterpret_cast<const uint8_t*>(p.depth_kv) +
                                 (((size_t(b) * Hk + hk) * nq + tile_qt(t)) * 2) * (size_t(kTileRows) * D * 2);
            for (int g0 = 0; g0 < p.l; g0 += kFwdDepthGroup) {
                const int gl = min(kFwdDepthGroup, p.l - g0);
                for (int kv = 0; kv < 2; ++kv)
                    for (int half = 0; half < NSUB; ++half)
                        for (int i = 0; i < gl; ++i, ++unit) {
                            const int st = unit % L::kRingStages;
                            if (unit >= L::kRingStages)
                                mbar_wait(bar(kBarDEmpty + st), ((unit / L::kRingStages) - 1) & 1, abort_flag, 32);
                            mbar_arrive_expect_tx(bar(kBarDFull + st), L::kUnitBytes);
                            bulk_load(sbase + L::kRing + st * L::kUnitBytes,
                                      blk + size_t(g0 + i) * slot_bytes + size_t(kv) * (size_t(kTileRows) * D * 2) + size_t(half) * L::kUnitBytes,
                                      L::kUnitBytes, bar(kBarDFull + st), policy);
                        }
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
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace moda
