// MoDA backward, fused form: five contractions and one exponential per score.
//
// The paper prints no backward pass; this is the derivative of the Sec. 2.2 operator.  With
// P = exp(S - LSE) (sequence), R = exp(U - LSE) (depth), D_t = <dO_t, O_t>:
//
//   dS = P o (dO V^T - D),   dU_i = R_i (<dO, Vd_i> - D)
//   dQ = scale (dS K + sum_i dU_i Kd_i)     dK = scale dS^T Q     dV = P^T dO
//   dKd_i = scale dU_i Q                    dVd_i = R_i dO        (row-local)
//
// Three launches on the caller's stream:
//   1. bwd_rows_kernel        everything that is local to a query row: D_t, and for every depth slot
//                             R_i, dU_i, dKd_i, dVd_i (written in cache layout) and the row's depth share
//                             of dQ, which initialises an fp32 dQ accumulator in the workspace.  Streams the
//                             depth cache exactly once; bound by HBM.
//   2. moda_bwd_fused_kernel  one CTA per 128-key tile, looping over the 128-query tiles at or below the
//                             diagonal.  Per pair of tiles: S^T = K Q^T and dP^T = V dO^T (tcgen05, operands
//                             in shared memory; one extra k-step each adds the per-query terms -LSE / scale and
//                             -D_t to every score of the query's column), P^T and dS^T formed once by the row warps, dV += P^T dO (P^T
//                             from tensor memory), dK += dS^T Q and dQ_tile = dS K (dS^T staged once in shared
//                             memory and used by both: K-major for dK, MN-major for dQ).  dK, dV accumulate in
//                             tensor memory over the whole loop; the dQ tile is added to the fp32 accumulator
//                             in L2 by bulk reductions (cp.reduce.async.bulk .add.f32) from a staging buffer --
//                             the only place where the order of floating-point additions depends on scheduling.
//   3. bwd_dq_finish_kernel   dQ = bf16(scale * accumulator).
//
// Against the split form (moda_bwd.cuh: a dQ pass and a dK/dV pass, seven contractions, every score
// exponentiated twice, bit-reproducible) this form does 5/7 of the tensor work and half of the
// exponentials; the host picks it unless the caller asks for reproducible bits.
#pragma once

#include "moda_bwd.cuh"
#include "moda_cache.cuh"
#include "moda_fwd.cuh"
#include "moda_fwd_wide.cuh"
#include "sm100_ptx.cuh"

namespace moda {

// fp32 dQ accumulator: [b][h][query tile][feature / 4][row 128][4], so that a warp whose lanes own
// consecutive rows adds (or stores) 512 contiguous bytes per instruction.
inline size_t dq_acc_bytes(int B, int T, int H, int d) {
    return size_t(B) * H * num_tiles(T) * kTileRows * d * 4;
}
// Workspace of the fused backward: row terms D_t, then the dQ accumulator (256-byte aligned).
inline size_t bwd_fused_rowterm_bytes(int B, int T, int H) {
    return (size_t(B) * H * T * 4 + 255) & ~size_t(255);
}
inline size_t bwd_fused_workspace_bytes(int B, int T, int H, int d) {
    return bwd_fused_rowterm_bytes(B, T, H) + dq_acc_bytes(B, T, H, d);
}

// =====================================================================================
// 1. Row-local part: D_t, depth gradients, depth share of dQ
// =====================================================================================
// One CTA per (b, h, 128-row tile); D / 32 threads per row, each owning 32 features (four 16-byte
// chunks of every depth row).  Lanes of a row are adjacent, so the two dot products of a slot are
// finished with shuffles; lanes with the same feature part own consecutive rows, so every warp access
// to the cache is a set of 128-byte (d = 128) or 256-byte (d = 64) runs.  q and dO stay packed in
// registers; a slot's key and value chunks are read once and used for everything the slot needs.
struct RowsParams {
    const __nv_bfloat16 *Q, *O, *dO;
    const void* depth_kv;   // bf16 cache, or e4m3 codes + row scales (FP8 instantiation); gradients are bf16 either way
    __nv_bfloat16* d_depth_kv;
    const float* LSE;
    float* delta;        // [B][H][T]
    float* dq_acc;       // accumulator layout above; every element is written (zeros when l == 0)
    int B, T, H, l;
    int accumulate;      // nonzero: depth gradients are added to d_depth_kv (bf16 adds in L2)
    float scale, scale_log2;
};

template <int D, bool FP8 = false>
__global__ void __launch_bounds__(kTileRows * (D / 32), 512 / (kTileRows * (D / 32)))
bwd_rows_kernel(const RowsParams p) {
    constexpr int PARTS = D / 32;                 // threads per row
    constexpr int CH = D / 8;                     // 16-byte chunks per row
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = lane % PARTS;
    const int r = warp * (32 / PARTS) + lane / PARTS;
    const int nq = num_tiles(p.T);
    const int qt = blockIdx.x % nq;
    const int bh = blockIdx.x / nq;
    const int b = bh / p.H, h = bh % p.H;
    const int t = qt * kTileRows + r;
    const bool valid = t < p.T;

    uint4 q4[4], g4[4];
    float dpart = 0.f;
    if (valid) {
        const size_t row = ((size_t(b) * p.T + t) * p.H + h) * CH + part * 4;
        const uint4* Q = reinterpret_cast<const uint4*>(p.Q) + row;
        const uint4* O = reinterpret_cast<const uint4*>(p.O) + row;
        const uint4* G = reinterpret_cast<const uint4*>(p.dO) + row;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            q4[j] = Q[j];
            g4[j] = G[j];
            dpart += dot8_bf16(O[j], g4[j]);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) q4[j] = g4[j] = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int off = 1; off < PARTS; off <<= 1) dpart += __shfl_xor_sync(0xffffffffu, dpart, off);
    const float delta = dpart;
    const size_t row_idx = (size_t(b) * p.H + h) * p.T + t;
    const float neg_lse2 = valid ? -p.LSE[row_idx] * kLog2e : -INFINITY;   // rows past T: R = 0, zero gradients
    if (valid && part == 0) p.delta[row_idx] = delta;

    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.f;

    if (FP8 && p.l > 0) {
        // e4m3 cache: this thread's 32 features are two 16-byte chunks of codes; the row's scale is one float per slot
        // for K and one for V.  Gradients are taken with respect to the dequantised keys and values.
        const size_t slot_stride = cache_slot_elems(p.B, p.T, p.H, D) / 8;                    // gradient cache, in uint4
        const size_t gblk = (size_t(bh) * nq + qt) * 2 * (kTileRows * CH) + size_t(part * 4) * kTileRows + r;
        uint4* gK = reinterpret_cast<uint4*>(p.d_depth_kv) + gblk;
        uint4* gV = gK + kTileRows * CH;
        const size_t slot_bytes8 = cache8_slot_bytes(p.B, p.T, p.H, D), blk_bytes8 = cache8_block_bytes(D);
        const uint8_t* cK = reinterpret_cast<const uint8_t*>(p.depth_kv) + (size_t(bh) * nq + qt) * 2 * blk_bytes8;
        const bool accumulate = p.accumulate != 0;
#pragma unroll 1
        for (int i = 0; i < p.l; ++i) {
            const uint8_t* cV = cK + blk_bytes8;
            uint4 k8[2], v8[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                k8[j] = __ldcs(reinterpret_cast<const uint4*>(cK) + size_t(part * 2 + j) * kTileRows + r);
                v8[j] = __ldcs(reinterpret_cast<const uint4*>(cV) + size_t(part * 2 + j) * kTileRows + r);
            }
            const float sk = __ldcs(reinterpret_cast<const float*>(cK + size_t(kTileRows) * D) + r);
            const float sv = __ldcs(reinterpret_cast<const float*>(cV + size_t(kTileRows) * D) + r);
            float kf[32];
            float u = 0.f, dr = 0.f;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t kw[4] = {k8[j].x, k8[j].y, k8[j].z, k8[j].w}, vw[4] = {v8[j].x, v8[j].y, v8[j].z, v8[j].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float v0, v1, v2, v3;
                    e4m3x4_to_f32(kw[k], kf[16 * j + 4 * k], kf[16 * j + 4 * k + 1], kf[16 * j + 4 * k + 2], kf[16 * j + 4 * k + 3]);
                    e4m3x4_to_f32(vw[k], v0, v1, v2, v3);
                    // features 16 j + 4 k .. + 3 of this thread = halves of the packed q / dO words 2 (4 j + k), 2 (4 j + k) + 1
                    const uint32_t* qw = reinterpret_cast<const uint32_t*>(q4) + 2 * (4 * j + k);
                    const uint32_t* gw = reinterpret_cast<const uint32_t*>(g4) + 2 * (4 * j + k);
                    u = fmaf(bf16_lo_to_f32(qw[0]), kf[16 * j + 4 * k], u);
                    u = fmaf(bf16_hi_to_f32(qw[0]), kf[16 * j + 4 * k + 1], u);
                    u = fmaf(bf16_lo_to_f32(qw[1]), kf[16 * j + 4 * k + 2], u);
                    u = fmaf(bf16_hi_to_f32(qw[1]), kf[16 * j + 4 * k + 3], u);
                    dr = fmaf(bf16_lo_to_f32(gw[0]), v0, dr);
                    dr = fmaf(bf16_hi_to_f32(gw[0]), v1, dr);
                    dr = fmaf(bf16_lo_to_f32(gw[1]), v2, dr);
                    dr = fmaf(bf16_hi_to_f32(gw[1]), v3, dr);
                }
            }
#pragma unroll
            for (int off = 1; off < PARTS; off <<= 1) {
                u += __shfl_xor_sync(0xffffffffu, u, off);
                dr += __shfl_xor_sync(0xffffffffu, dr, off);
            }
            const float R = fast_exp2(fmaf(u * sk, p.scale_log2, neg_lse2));
            const float dU = R * (dr * sv - delta);
            const uint32_t r2 = pack_bf16x2(R, R);
            const float sdu = dU * p.scale;
            const uint32_t sdu2 = pack_bf16x2(sdu, sdu);
            const float duk = dU * sk;                        // dQ share: dU * (scale_k * code)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 ov, ok;
                ov.x = mul_bf16x2(g4[j].x, r2); ov.y = mul_bf16x2(g4[j].y, r2);
                ov.z = mul_bf16x2(g4[j].z, r2); ov.w = mul_bf16x2(g4[j].w, r2);
                ok.x = mul_bf16x2(q4[j].x, sdu2); ok.y = mul_bf16x2(q4[j].y, sdu2);
                ok.z = mul_bf16x2(q4[j].z, sdu2); ok.w = mul_bf16x2(q4[j].w, sdu2);
                if (accumulate) {
                    red_add_bf16x2_v4(gV + j * kTileRows, ov);
                    red_add_bf16x2_v4(gK + j * kTileRows, ok);
                } else {
                    __stcs(gV + j * kTileRows, ov);
                    __stcs(gK + j * kTileRows, ok);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[8 * j + e] = fmaf(duk, kf[8 * j + e], acc[8 * j + e]);
            }
            cK += slot_bytes8; gK += slot_stride; gV += slot_stride;
        }
    } else
    if (p.l > 0) {
        const size_t slot_stride = cache_slot_elems(p.B, p.T, p.H, D) / 8;                    // in uint4
        const size_t blk = (size_t(bh) * nq + qt) * 2 * (kTileRows * CH) + size_t(part * 4) * kTileRows + r;
        const uint4* cK = reinterpret_cast<const uint4*>(p.depth_kv) + blk;
        const uint4* cV = cK + kTileRows * CH;
        uint4* gK = reinterpret_cast<uint4*>(p.d_depth_kv) + blk;
        uint4* gV = gK + kTileRows * CH;
        const bool accumulate = p.accumulate != 0;
#pragma unroll 1
        for (int i = 0; i < p.l; ++i) {
            uint4 kc[4], vc[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                kc[j] = __ldcs(cK + j * kTileRows);          // streamed: every byte of the cache is used once
                vc[j] = __ldcs(cV + j * kTileRows);
            }
            float u = 0.f, dr = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                u += dot8_bf16(q4[j], kc[j]);
                dr += dot8_bf16(g4[j], vc[j]);
            }
#pragma unroll
            for (int off = 1; off < PARTS; off <<= 1) {
                u += __shfl_xor_sync(0xffffffffu, u, off);
                dr += __shfl_xor_sync(0xffffffffu, dr, off);
            }
            const float R = fast_exp2(fmaf(u, p.scale_log2, neg_lse2));   // the forward's LSE covers both key sets
            const float dU = R * (dr - delta);
            const uint32_t r2 = pack_bf16x2(R, R);
            const float sdu = dU * p.scale;
            const uint32_t sdu2 = pack_bf16x2(sdu, sdu);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 ov, ok;
                ov.x = mul_bf16x2(g4[j].x, r2); ov.y = mul_bf16x2(g4[j].y, r2);
                ov.z = mul_bf16x2(g4[j].z, r2); ov.w = mul_bf16x2(g4[j].w, r2);
                ok.x = mul_bf16x2(q4[j].x, sdu2); ok.y = mul_bf16x2(q4[j].y, sdu2);
                ok.z = mul_bf16x2(q4[j].z, sdu2); ok.w = mul_bf16x2(q4[j].w, sdu2);
                if (accumulate) {
                    red_add_bf16x2_v4(gV + j * kTileRows, ov);
                    red_add_bf16x2_v4(gK + j * kTileRows, ok);
                } else {
                    __stcs(gV + j * kTileRows, ov);
                    __stcs(gK + j * kTileRows, ok);
                }
                acc[8 * j + 0] = fmaf(dU, bf16_lo_to_f32(kc[j].x), acc[8 * j + 0]);
                acc[8 * j + 1] = fmaf(dU, bf16_hi_to_f32(kc[j].x), acc[8 * j + 1]);
                acc[8 * j + 2] = fmaf(dU, bf16_lo_to_f32(kc[j].y), acc[8 * j + 2]);
                acc[8 * j + 3] = fmaf(dU, bf16_hi_to_f32(kc[j].y), acc[8 * j + 3]);
                acc[8 * j + 4] = fmaf(dU, bf16_lo_to_f32(kc[j].z), acc[8 * j + 4]);
                acc[8 * j + 5] = fmaf(dU, bf16_hi_to_f32(kc[j].z), acc[8 * j + 5]);
                acc[8 * j + 6] = fmaf(dU, bf16_lo_to_f32(kc[j].w), acc[8 * j + 6]);
                acc[8 * j + 7] = fmaf(dU, bf16_hi_to_f32(kc[j].w), acc[8 * j + 7]);
            }
            cK += slot_stride; cV += slot_stride; gK += slot_stride; gV += slot_stride;
        }
    }
    // depth share of dQ (unscaled) -> accumulator; the fused kernel adds the sequence share on top
    float4* dst = reinterpret_cast<float4*>(p.dq_acc) + (size_t(bh) * nq + qt) * (D / 4) * kTileRows + size_t(part * 8) * kTileRows + r;
#pragma unroll
    for (int j = 0; j < 8; ++j)
        dst[j * kTileRows] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
}

// =====================================================================================
// 3. dQ = bf16(scale * accumulator)
// =====================================================================================
template <int D>
__global__ void __launch_bounds__(kTileRows * (D / 32))
bwd_dq_finish_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dQ, int B, int T, int H, float scale) {
    constexpr int PARTS = D / 32;
    constexpr int CH = D / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = lane % PARTS;
    const int r = warp * (32 / PARTS) + lane / PARTS;
    const int nq = num_tiles(T);
    const int qt = blockIdx.x % nq;
    const int bh = blockIdx.x / nq;
    const int b = bh / H, h = bh % H;
    const int t = qt * kTileRows + r;
    if (t >= T) return;
    const float4* src = reinterpret_cast<const float4*>(dq_acc) + size_t(blockIdx.x) * (D / 4) * kTileRows + size_t(part * 8) * kTileRows + r;
    uint4* dst = reinterpret_cast<uint4*>(dQ) + ((size_t(b) * T + t) * H + h) * CH + part * 4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float4 a = __ldcs(src + (2 * j) * kTileRows);
        const float4 c = __ldcs(src + (2 * j + 1) * kTileRows);
        uint4 o;
        o.x = pack_bf16x2(a.x * scale, a.y * scale); o.y = pack_bf16x2(a.z * scale, a.w * scale);
        o.z = pack_bf16x2(c.x * scale, c.y * scale); o.w = pack_bf16x2(c.z * scale, c.w * scale);
        dst[j] = o;
    }
}

// =====================================================================================
// 2. Sequence part: dK, dV and the dQ tiles
// =====================================================================================
// 512 threads (in warp order):
//   row warps    two warpgroups: a thread owns one key row (= tensor-memory lane) and 64 of the 128 query columns of
//                an iteration: P^T, then dS^T.
//   drain warps  one warpgroup: a thread owns one query row of the dQ tile; it copies the row out of tensor memory
//                (which frees the region at once) and hands it, 8 KiB at a time through a staging ring in shared
//                memory, to bulk reductions into the fp32 accumulator, at whatever pace L2 takes them, without
//                holding up the row warps.
//   then         a loader warp (TMA tiles; the per-query terms as bf16 parts for the extra k-step) and the warps
//                that issue the contractions:
//                S, dP, and dV then dQ then dK.  One tcgen05.mma costs its
//                issuing thread about as long as it executes, so the contractions that start an iteration's two
//                chains have their own warps on different schedulers; MMAs of different warps are ordered by
//                mbarriers only.
//
// Tensor memory (fp32 columns): X, 128 columns per buffer, S^T overlaid by P^T (bf16) -- one buffer at d = 128,
// two at d = 64 (where dK and dV leave room);  Y, 128 columns, dP^T and then the dQ tile of the same iteration;
// dK, D columns;  dV, D columns.  512 columns at either head width.
//
// What bounds it (cycle stamps per warp role, T = 8192): the rate at which a dQ tile's additions are taken by L2 (64 KiB
// of fp32 per iteration per SM at d = 128; all SMs together sustain about 5.9 TB/s in a kernel that does nothing else,
// 4.3 TB/s here beside as many bytes of Q / dO loads): the drain warps need ~4300 cycles per tile, the five contractions
// 2700 tensor cycles.  The shared-memory port (MMA operands 304 KiB per iteration, TMA writes 64 KiB, dS^T 32 KiB, the
// dQ staging 64 KiB in and out, against 128 bytes per clock) is at two thirds of its peak since the row warps no
// longer load the per-query terms.
//
// Two dependency chains per iteration i, which overlap each other and the next iteration:
//   X:  S'_i = S_i - LSE / scale -> P_i^T = exp2(S' c) (row warps) -> dV_i -> X free -> S_{i+1}
//   Y:  dP'_i = dP_i - D -> dS_i^T = P o dP' to shared memory (row warps) -> dQ_i -> copied out (drain warps) -> Y free -> dP_{i+1}
// and dK_i, issued behind dQ_i, fills the tensor pipe while the row warps exponentiate tile i+1.

template <int D>
struct FusedSmem {
    static constexpr int kRowWGs = 2;                          // row warpgroups (64 query columns per thread)
    static constexpr int kCols = kTileRows / kRowWGs;          // query columns per row-warp thread
    static constexpr int kThreads = (kRowWGs * 4 + 8) * 32;    // row warps, 4 drain warps, loader + 3 issuers
    static constexpr int kTileBytes = kTileRows * D * 2;       // 128 x D bf16
    static constexpr int kSubBytes = kTileRows * 128;          // 128 x 64 sub-tile (128-byte rows)
    // Stages of Q_i.  Q_i is read by S_i early and by dK_i late in its iteration, and a tile takes about 1600
    // cycles from the TMA issue to the first MMA that uses it, so with two stages the chain "dK_{i-2} completes ->
    // load Q_i -> S_i -> P_i -> dS_i -> dK_i" spans two iterations and sets the pace; three stages (d = 64, where
    // shared memory has room) take the load off that chain.
    static constexpr int kStages = (D == 64) ? 3 : 2;
    // dO_i is read by dP_i and dV_i, both of which complete before dP_{i+1} can be issued; at d = 128 one
    // stage leaves the 32 KiB that the dQ staging buffer needs
    static constexpr int kdOStages = (D == 128) ? 1 : 2;
    static constexpr int kK = 0;
    static constexpr int kV = kK + kTileBytes;
    static constexpr int kQ = kV + kTileBytes;                 // stages of Q_i
    static constexpr int kdO = kQ + kStages * kTileBytes;      // stages of dO_i
    static constexpr int kdS = kdO + kdOStages * kTileBytes;   // dS^T: 128 keys x 128 queries bf16
    static constexpr int kdSBytes = kTileRows * kTileRows * 2;
    static constexpr int kStg = kdS + kdSBytes;                // ring of 8 KiB chunks (16 feature columns of a dQ tile, fp32, accumulator layout)
    static constexpr int kStgSlots = (D == 128) ? 3 : 4;       // three measured as fast as four; two cost 3-4 %
    static constexpr int kStgBytes = kStgSlots * 16 * kTileRows * 4;
    // Operands of the extra k-step that adds the per-query terms to the two score contractions (see the kernel):
    // 2 KiB chunks of [128 rows][8 bf16] (unswizzled core matrices, 16 bytes per row): one per Q stage with the
    // stage's terms, then the two constant "ones" chunks and a zero chunk.
    static constexpr int kAug = kStg + kStgBytes;
    static constexpr int kAugChunk = kTileRows * 16;
    static constexpr int kAugOnesS = kAug + kStages * kAugChunk;
    static constexpr int kAugOnesD = kAugOnesS + kAugChunk;
    static constexpr int kAugZero = kAugOnesD + kAugChunk;
    static constexpr int kBars = kAugZero + kAugChunk;
    static constexpr int kNumBars = 28;
    static constexpr int kMisc = kBars + kNumBars * 8;
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kSmemLimit = 232448;                  // 227 KiB per CTA on sm_100
    // the tiles need a 1024-byte aligned base; ask for the slack when it fits (d = 64), else rely on the
    // dynamic segment starting aligned and check at run time (aligned_dynamic_smem)
    static constexpr int kDynamic = (kTotal + 1024 <= kSmemLimit) ? kTotal + 1024 : kSmemLimit;
    static_assert(kTotal <= kSmemLimit, "shared-memory plan too large");
};

enum FusedBar : int {
    kFBarKV = 0,
    kFBarQFull = 1,     // +stage (<= 3), count 32: Q_i and the per-query terms of the stage have landed
    kFBarQEmpty = 4,    // +stage (<= 3): dK_i complete (Q_i, the row terms and the dS buffer are free)
    kFBardOFull = 7,    // +stage (<= 2)
    kFBardOEmpty = 9,   // +stage (<= 2), count 2: dP_i and dV_i complete
    kFBarSFull = 11,    // +X buffer: S_i complete
    kFBarPFull = 13,    // +X buffer, count 256: P_i^T written
    kFBardPFull = 15,   // dP_i complete
    kFBardSFull = 16,   // count 256: dS_i^T written to shared memory, dP_i consumed
    kFBarXFree = 17,    // +X buffer: dV_i complete: the buffer may take S_{i + buffers}
    kFBardQFull = 19,   // dQ_i complete
    kFBarYFree = 20,    // count 128: dQ_i copied out: Y may take dP_{i+1}
    kFBarFinal = 21,    // last dV and dK complete (one warp issues both)
    kFBarDrain = 22,    // +issuer (3): abort path only
};

struct FusedParams {
    const float* LSE;
    const float* delta;
    float* dq_acc;
    int B, T, H;        // H = number of query heads
    int G;              // query heads per key/value head; dK, dV sum over the G heads of a group
    float scale, scale_log2;
};

template <int D>
__global__ void __launch_bounds__(FusedSmem<D>::kThreads, 1)
moda_bwd_fused_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                      const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
                      const __grid_constant__ CUtensorMap mapdK, const __grid_constant__ CUtensorMap mapdV,
                      const FusedParams p) {
    using L = FusedSmem<D>;
    constexpr int NSUB = D / 64;
    constexpr int NRW = L::kRowWGs, COLS = L::kCols, NROW = 128 * NRW;      // row warpgroups, columns per thread, row threads
    constexpr int W_DRAIN = 4 * NRW, W_LOAD = W_DRAIN + 4, W_S = W_LOAD + 1, W_DP = W_LOAD + 2;
    constexpr int W_ACC = W_LOAD + 3;                             // issues the three accumulating contractions
    constexpr int NOTHER = (L::kThreads / 32 - W_LOAD) * 32;      // threads of the loader / issuer warps
    constexpr uint32_t kTmemCols = 512;
    // d = 64 leaves room for a second S^T / P^T buffer: S_{i+1} is then computed while the row warps still work
    // on tile i, instead of waiting for dV_i to release the only buffer.
    constexpr int XB = (D == 64) ? 2 : 1;
    constexpr uint32_t kColX = 0, kColY = 128 * XB, kColdK = kColY + 128, kColdV = kColdK + D;
    static_assert(kColdV + D <= kTmemCols, "tensor-memory plan too large");

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
    auto bar = [&](int i) { return sbase + L::kBars + 8u * uint32_t(i); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nk = num_tiles(p.T);
    const int bh = blockIdx.x / nk;
    const int kt = blockIdx.x % nk;                       // key tiles in ascending order: most work first
    const int Hk = p.H / p.G;
    const int b = bh / Hk, h = bh % Hk;                   // h: key/value head of this CTA
    const int k0 = kt * kTileRows;
    const int n_per = nk - kt;                            // query tiles kt .. nk-1 see this key tile
    const int n_it = n_per * p.G;                         // iteration it: query head h G + it / n_per, tile kt + it % n_per

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(kFBarKV), 1);
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(bar(kFBarQFull + s), 32);
            mbar_init(bar(kFBarQEmpty + s), 1);
        }
        for (int s = 0; s < L::kdOStages; ++s) {
            mbar_init(bar(kFBardOFull + s), 1);
            mbar_init(bar(kFBardOEmpty + s), 2);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kFBarSFull + s), 1);
            mbar_init(bar(kFBarPFull + s), NROW);
            mbar_init(bar(kFBarXFree + s), 1);
        }
        mbar_init(bar(kFBardPFull), 1);
        mbar_init(bar(kFBardSFull), NROW);
        mbar_init(bar(kFBardQFull), 1);
        mbar_init(bar(kFBarYFree), 128);
        mbar_init(bar(kFBarFinal), 1);
        for (int s = 0; s < 3; ++s) mbar_init(bar(kFBarDrain + s), 1);
        fence_mbar_init();
    }
    if (warp == W_S) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    {   // constant chunks of the extra k-step: 1.0 in columns 0-2 (S) / 4-6 (dP), zero elsewhere; the per-stage chunks start
        // at zero because the chunk behind the one in use is read too (against the zero chunk: it only has to be finite)
        constexpr uint32_t kOne2 = 0x3F803F80u, kOne1 = 0x00003F80u;
        uint4* aug = reinterpret_cast<uint4*>(smem + L::kAug);
        for (int i = threadIdx.x; i < (L::kStages + 3) * kTileRows; i += L::kThreads) {
            const int chunk = i / kTileRows;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (chunk == L::kStages) v = make_uint4(kOne2, kOne1, 0u, 0u);
            if (chunk == L::kStages + 1) v = make_uint4(0u, 0u, kOne2, kOne1);
            aug[i] = v;
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    // Abort path of an issuing thread: wait (bounded) until its own MMAs have drained.
    auto drain_on_abort = [&](int which) {
        if (*abort_flag != 0) {
            umma_commit(bar(kFBarDrain + which));
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(bar(kFBarDrain + which), 0) && globaltimer_ns() - t0 < 20000000ull) {}
        }
    };

    // Register budget: the CTA owns what it was launched with (512 threads x 128 registers), and setmaxnreg.inc blocks until the CTA's own pool can serve it, so the three shares must fit that total.
    constexpr int kRegsLaunch = 128;
    static_assert(L::kThreads == 512, "the register shares below assume 512 threads");
    // Shares measured (T = 8192 .. 65536): the issuing warps need about 100 registers to keep their descriptors and
    // barrier addresses without spills; d = 128: 128 / 160 / 96 (42.1 ms at T = 65536 against 44.1 with 136 / 160 / 80),
    // d = 64: 136 / 136 / 104 (27.6 ms at T = 32768, H = 32 against 28.5 with 152 / 152 / 56).
    constexpr int kRegsRow = (D == 128) ? 128 : 136, kRegsDrain = (D == 128) ? 160 : 136, kRegsOther = (D == 128) ? 96 : 104;
    static_assert(NROW * kRegsRow + 128 * kRegsDrain + NOTHER * kRegsOther <= L::kThreads * kRegsLaunch, "register shares exceed the CTA's pool");
    // setmaxnreg.inc to less than the current count (or .dec to more) is an illegal instruction
    static_assert(kRegsRow >= kRegsLaunch && kRegsDrain >= kRegsLaunch && kRegsOther <= kRegsLaunch, "setmaxnreg direction");
    if (warp < W_DRAIN) {
        // =========================== row warps: P^T, dS^T, dK / dV epilogue ===========================
        setmaxnreg_inc<kRegsRow>();
        const int hc = warp >> 2;                            // which COLS query columns of every iteration
        const int r = tid & 127;                             // key row inside the tile = TMEM lane
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        const uint32_t tX0 = tmem + lane_addr + kColX + hc * COLS;
        const uint32_t tY = tmem + lane_addr + kColY + hc * COLS;
        // this thread's row of dS^T: sub-tile of its 64-column half, 128-byte rows, its first 16-byte chunk
        uint8_t* ds_row = smem + L::kdS + ((hc * COLS) >> 6) * L::kSubBytes + r * 128;
        const int ds_chunk0 = ((hc * COLS) & 63) >> 3;
        for (int it = 0; it < n_it; ++it) {
            const int st = it % L::kStages;
            const bool diag = (it % n_per) == 0;             // the query tile is the key tile itself: causal mask
            uint32_t pk[COLS / 2];                           // P_i^T of this thread: COLS values, bf16 pairs
            // ---- P_i^T ----
            const int xb = it % XB;
            const uint32_t tX = tX0 + xb * 128;
            mbar_wait(bar(kFBarSFull + xb), (it / XB) & 1, abort_flag, 121);
            tc_fence_after_sync();
            {
                // all blocks are requested before the first is used: the later loads' latency hides under the
                // first block's exponentials
                uint32_t sv[COLS];
#pragma unroll
                for (int c = 0; c < COLS / 32; ++c) tmem_ld32(tX + c * 32, *reinterpret_cast<uint32_t(*)[32]>(sv + c * 32));
                tmem_wait_ld();
#pragma unroll
                for (int i4 = 0; i4 < COLS / 4; ++i4) {
                    // the contraction has already subtracted LSE / scale from every score of the query's column
                    float e0 = fast_exp2(__uint_as_float(sv[4 * i4 + 0]) * p.scale_log2);
                    float e1 = fast_exp2(__uint_as_float(sv[4 * i4 + 1]) * p.scale_log2);
                    float e2 = fast_exp2(__uint_as_float(sv[4 * i4 + 2]) * p.scale_log2);
                    float e3 = fast_exp2(__uint_as_float(sv[4 * i4 + 3]) * p.scale_log2);
                    if (diag) {                               // query column c sees key row r iff c >= r
                        const int c = hc * COLS + 4 * i4;
                        if (c + 0 < r) e0 = 0.f;
                        if (c + 1 < r) e1 = 0.f;
                        if (c + 2 < r) e2 = 0.f;
                        if (c + 3 < r) e3 = 0.f;
                    }
                    pk[2 * i4] = pack_bf16x2(e0, e1);
                    pk[2 * i4 + 1] = pack_bf16x2(e2, e3);
                }
            }
            // P^T (bf16, two per column) overlays the first half of the columns this thread has read
            if constexpr (COLS == 64) tmem_st32(tX, *reinterpret_cast<uint32_t(*)[32]>(pk));
            else tmem_st16(tX, *reinterpret_cast<uint32_t(*)[16]>(pk));
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(kFBarPFull + xb));

            // ---- dS_i^T = P o (dP - D), with the bf16 P that dV uses ----
            mbar_wait(bar(kFBardPFull), it & 1, abort_flag, 122);
            tc_fence_after_sync();
            // the dS buffer is still read by dQ_{i-1} and dK_{i-1} (dK is issued last: its completion covers both)
            if (it > 0) mbar_wait(bar(kFBarQEmpty + (it - 1) % L::kStages), ((it - 1) / L::kStages) & 1, abort_flag, 123);
            {
                uint32_t gv[COLS];
#pragma unroll
                for (int c = 0; c < COLS / 32; ++c) tmem_ld32(tY + c * 32, *reinterpret_cast<uint32_t(*)[32]>(gv + c * 32));
                tmem_wait_ld();
#pragma unroll
                for (int g = 0; g < COLS / 8; ++g) {         // 8 query columns = one 16-byte chunk of the row
                    const uint32_t* pp = pk + 4 * g;         // gv holds dP - D_t already (subtracted by the contraction)
                    uint4 v;
                    v.x = pack_bf16x2(bf16_lo_to_f32(pp[0]) * __uint_as_float(gv[8 * g + 0]),
                                      bf16_hi_to_f32(pp[0]) * __uint_as_float(gv[8 * g + 1]));
                    v.y = pack_bf16x2(bf16_lo_to_f32(pp[1]) * __uint_as_float(gv[8 * g + 2]),
                                      bf16_hi_to_f32(pp[1]) * __uint_as_float(gv[8 * g + 3]));
                    v.z = pack_bf16x2(bf16_lo_to_f32(pp[2]) * __uint_as_float(gv[8 * g + 4]),
                                      bf16_hi_to_f32(pp[2]) * __uint_as_float(gv[8 * g + 5]));
                    v.w = pack_bf16x2(bf16_lo_to_f32(pp[3]) * __uint_as_float(gv[8 * g + 6]),
                                      bf16_hi_to_f32(pp[3]) * __uint_as_float(gv[8 * g + 7]));
                    *reinterpret_cast<uint4*>(ds_row + (((ds_chunk0 + g) ^ (r & 7)) << 4)) = v;
                }
            }
            fence_proxy_async_smem();                        // generic-proxy stores -> read by the MMAs (async proxy)
            tc_fence_before_sync();
            mbar_arrive(bar(kFBardSFull));
        }

        // ---- epilogue: dK (scaled) by the first warpgroup, dV by the second ----
        if (hc < 2) {
        mbar_wait(bar(kFBarFinal), 0, abort_flag, 124);
        tc_fence_after_sync();
        {
            const float mul = hc == 0 ? p.scale : 1.f;
            const uint32_t col = hc == 0 ? kColdK : kColdV;
            const int dst_off = hc == 0 ? L::kQ : L::kdO;    // every MMA has completed: the stages are free
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
                tma_store_4d(&mapdK, sbase + L::kQ + s * L::kSubBytes, s * 64, h, k0, b);
                tma_store_4d(&mapdV, sbase + L::kdO + s * L::kSubBytes, s * 64, h, k0, b);
            }
            tma_store_commit();
            tma_store_wait_all();
        }
        }
    } else if (warp < W_LOAD) {
        // =========================== drain warps: dQ tile -> fp32 accumulator ===========================
        // The tile leaves the SM as bulk reductions (cp.reduce.async.bulk, fp32 add in L2) from a staging buffer
        // in shared memory.  Per-thread red.global instructions would do the same additions, but they queue in the
        // load/store path of the SM at the pace L2 takes them, and every shared-memory load, store and barrier probe of
        // the row warps then waits behind them (measured: + 2000 cycles per iteration).
        setmaxnreg_inc<kRegsDrain>();
        const int r = tid & 127;                             // query row inside the tile = TMEM lane
        const uint32_t tY = tmem + (uint32_t((warp & 3) * 32) << 16) + kColY;
        float4* stg = reinterpret_cast<float4*>(smem + L::kStg) + r;          // [feature / 4 (16)][row 128] float4
        for (int it = 0; it < n_it; ++it) {
            const int hq = h * p.G + it / n_per;
            const int qi = kt + it % n_per;
            float* dst = p.dq_acc + ((size_t(b) * p.H + hq) * nk + qi) * (size_t(kTileRows) * D);
            mbar_wait(bar(kFBardQFull), it & 1, abort_flag, 120);
            tc_fence_after_sync();
            uint32_t o[D];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) tmem_ld32(tY + c * 32, *reinterpret_cast<uint32_t(*)[32]>(o + c * 32));
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(bar(kFBarYFree));                    // Y may take dP of the next iteration
            // 16 feature columns (8 KiB, contiguous in the accumulator) at a time through a ring of staging chunks:
            // a chunk is rewritten once the reduction issued from it one ring earlier has finished reading it, so
            // all but one of the ring's reductions stay in flight and L2, not this loop, sets the pace.
#pragma unroll
            for (int ch = 0; ch < D / 16; ++ch) {
                const int slot = (it * (D / 16) + ch) % L::kStgSlots;      // the ring runs on across iterations
                if (tid == NROW) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(L::kStgSlots - 1) : "memory");
                asm volatile("bar.sync 2, 128;" ::: "memory");
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    stg[(slot * 4 + g) * kTileRows] = make_float4(__uint_as_float(o[ch * 16 + 4 * g]), __uint_as_float(o[ch * 16 + 4 * g + 1]),
                                                                  __uint_as_float(o[ch * 16 + 4 * g + 2]), __uint_as_float(o[ch * 16 + 4 * g + 3]));
                fence_proxy_async_smem();
                asm volatile("bar.sync 2, 128;" ::: "memory");
                if (tid == NROW) {
                    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
                                 ::"l"(dst + ch * (16 * kTileRows)), "r"(sbase + L::kStg + slot * (16 * kTileRows * 4)), "r"(16 * kTileRows * 4) : "memory");
                    tma_store_commit();
                }
            }
        }
        if (tid == NROW) tma_store_wait_all();               // every addition has been performed before the CTA retires
    } else {
      setmaxnreg_dec<kRegsOther>();
      if (warp == W_LOAD) {
        // =========================== loader: TMA tiles + per-query LSE, D_t ===========================
        if (lane == 0) {
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapdO);
            mbar_arrive_expect_tx(bar(kFBarKV), 2 * L::kTileBytes);
#pragma unroll
            for (int s = 0; s < NSUB; ++s) {
                tma_load_4d(sbase + L::kK + s * L::kSubBytes, &mapK, bar(kFBarKV), s * 64, h, k0, b);
                tma_load_4d(sbase + L::kV + s * L::kSubBytes, &mapV, bar(kFBarKV), s * 64, h, k0, b);
            }
        }
        const float inv_scale = 1.f / p.scale;
        for (int it = 0; it < n_it; ++it) {
            const int st = it % L::kStages;
            const int hq = h * p.G + it / n_per;
            const size_t row_base = (size_t(b) * p.H + hq) * p.T;
            const int qrow0 = (kt + it % n_per) * kTileRows;
            // lane handles query columns 4 lane .. 4 lane + 3: for each, -LSE / scale and -D_t as three bf16 parts
            // (hi + mid + lo = the fp32 value); queries past T get a large negative first term so that P = 0
            uint4 av[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = qrow0 + 4 * lane + j;
                const float nl = (c < p.T) ? -p.LSE[row_base + c] * inv_scale : -1.0e30f;
                const float nd = (c < p.T) ? -p.delta[row_base + c] : 0.f;
                av[j] = make_uint4(0u, 0u, 0u, 0u);
                split3_bf16(nl, av[j].x, av[j].y);
                split3_bf16(nd, av[j].z, av[j].w);
            }
            if (it >= L::kStages) mbar_wait(bar(kFBarQEmpty + st), ((it - L::kStages) / L::kStages) & 1, abort_flag, 130);
            uint4* aug = reinterpret_cast<uint4*>(smem + L::kAug + st * L::kAugChunk) + 4 * lane;
#pragma unroll
            for (int j = 0; j < 4; ++j) aug[j] = av[j];
            fence_proxy_async_smem();                        // generic-proxy stores -> read by the MMAs (async proxy)
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(kFBarQFull + st), L::kTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s)
                    tma_load_4d(sbase + L::kQ + st * L::kTileBytes + s * L::kSubBytes, &mapQ, bar(kFBarQFull + st), s * 64, hq, qrow0, b);
                const int dst = it % L::kdOStages;
                if (it >= L::kdOStages) mbar_wait(bar(kFBardOEmpty + dst), ((it - L::kdOStages) / L::kdOStages) & 1, abort_flag, 131);
                mbar_arrive_expect_tx(bar(kFBardOFull + dst), L::kTileBytes);
#pragma unroll
                for (int s = 0; s < NSUB; ++s)
                    tma_load_4d(sbase + L::kdO + dst * L::kTileBytes + s * L::kSubBytes, &mapdO, bar(kFBardOFull + dst), s * 64, hq, qrow0, b);
            } else {
                mbar_arrive(bar(kFBarQFull + st));
            }
        }
      } else if (warp == W_S || warp == W_DP) {
        // ============ MMA issuers: S^T = K Q^T (warp 13, into X), dP^T = V dO^T (warp 14, into Y) ============
        {   // whole warp: operands are warp-uniform, one elected lane issues
            const bool is_s = (warp == W_S);
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
            const uint32_t a_tile = sbase + (is_s ? L::kK : L::kV);
            const int full0 = is_s ? kFBarQFull : kFBardOFull;
            const int nb = is_s ? XB : 1;                                 // accumulator buffers of this contraction
            // a descriptor of a later k-step is the first one plus a compile-time constant (the start-address field
            // counts 16-byte units and stays inside its 14 bits below 256 KiB)
            const uint64_t da0 = desc_kmajor_sw128(a_tile, 0);
            const uint64_t db0 = desc_kmajor_sw128(sbase + (is_s ? L::kQ : L::kdO), 0);
            // extra k-step: A = ones in the columns of this contraction's terms (second k-chunk: the zero chunk),
            // B = the Q stage's chunk of per-query terms (second k-chunk: whatever follows it, finite, times zero)
            const uint64_t da_aug = make_smem_desc_noswz(sbase + (is_s ? L::kAugOnesS : L::kAugOnesD),
                                                         uint32_t(L::kAugZero - (is_s ? L::kAugOnesS : L::kAugOnesD)), 128u);
            const uint64_t db_aug0 = make_smem_desc_noswz(sbase + L::kAug, uint32_t(L::kAugChunk), 128u);
            mbar_wait(bar(kFBarKV), 0, abort_flag, 140);
            const int nst = is_s ? L::kStages : L::kdOStages;
            for (int it = 0; it < n_it; ++it) {
                const int st = it % nst;
                // the accumulator buffer still holds P of its previous tile (until that dV completes) / dQ_{i-1} (until
                // it is copied out)
                const int xb = it % nb;
                const uint32_t col = is_s ? kColX + xb * 128 : kColY;
                const uint32_t free_bar = is_s ? bar(kFBarXFree + xb) : bar(kFBarYFree);
                if (it >= nb) mbar_wait2(bar(full0 + st), (it / nst) & 1, free_bar, ((it - nb) / nb) & 1, abort_flag, 141, is_s ? 142 : 143);
                else mbar_wait(bar(full0 + st), (it / nst) & 1, abort_flag, 141);
                // dP also needs the Q stage's per-query terms (they arrive with Q_i)
                const int qst = it % L::kStages;
                if (!is_s) mbar_wait(bar(kFBarQFull + qst), (it / L::kStages) & 1, abort_flag, 147);
                tc_fence_after_sync();
                const uint64_t db = db0 + uint64_t((st * L::kTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    umma_ss(tmem + col, da0 + uint64_t(((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4),
                            db + uint64_t(((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4), idesc_s, kk > 0);
                umma_ss(tmem + col, da_aug, db_aug0 + uint64_t((qst * L::kAugChunk) >> 4), idesc_s, 1u);
                umma_commit(bar(is_s ? kFBarSFull + xb : kFBardPFull));
                if (!is_s) umma_commit(bar(kFBardOEmpty + st));
            }
            drain_on_abort(is_s ? 0 : 1);
        }
      } else if (warp == W_ACC) {
        // ============ MMA issuer of the accumulating contractions: dV_i += P^T dO (P^T from tensor memory, dO MN-major),
        // ============ then, once dS_i^T is in shared memory, dQ_tile = dS K into Y (dS^T and K both MN-major) and
        // ============ dK += dS^T Q (dS^T K-major, Q MN-major).  P_i, dS_i, P_{i+1} are produced in this order, so one
        // ============ warp can take the three in turn.  dQ before dK: its tile has to be copied out before dP of the next
        // ============ iteration can land, dK only has to finish before dS_{i+1} is written.  (A warp per contraction was
        // ============ measured at d = 64, where these are N = 64 MMAs: no faster.)
        {
            constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, false, true);
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, true, true);
            const uint64_t dvb0 = desc_mnmajor_sw128(sbase + L::kdO, 0, L::kSubBytes);
            const uint64_t dqa0 = desc_mnmajor_sw128(sbase + L::kdS, 0, L::kSubBytes);
            const uint64_t dqb0 = desc_mnmajor_sw128(sbase + L::kK, 0, L::kSubBytes);
            const uint64_t dka0 = desc_kmajor_sw128(sbase + L::kdS, 0);
            const uint64_t dkb0 = desc_mnmajor_sw128(sbase + L::kQ, 0, L::kSubBytes);
            for (int it = 0; it < n_it; ++it) {
                const int st = it % L::kStages, dst = it % L::kdOStages, xb = it % XB;
                mbar_wait2(bar(kFBarPFull + xb), (it / XB) & 1, bar(kFBardOFull + dst), (it / L::kdOStages) & 1, abort_flag, 144, 145);
                tc_fence_after_sync();
                const uint64_t dvb = dvb0 + uint64_t((dst * L::kTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < kTileRows / 16; ++kk)  // 16 queries per k-step: 8 columns, in the block of the row warpgroup that owns them
                    umma_ts(tmem + kColdV, tmem + kColX + xb * 128 + (kk / (COLS / 16)) * COLS + (kk % (COLS / 16)) * 8, dvb + uint64_t(kk * 128),
                            idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar(kFBarXFree + xb));
                umma_commit(bar(kFBardOEmpty + dst));
                mbar_wait(bar(kFBardSFull), it & 1, abort_flag, 146);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kTileRows / 16; ++kk)
                    umma_ss(tmem + kColY, dqa0 + uint64_t(kk * 128), dqb0 + uint64_t(kk * 128), idesc_dq, kk > 0);
                umma_commit(bar(kFBardQFull));
                const uint64_t dkb = dkb0 + uint64_t((st * L::kTileBytes) >> 4);
#pragma unroll
                for (int kk = 0; kk < kTileRows / 16; ++kk)
                    umma_ss(tmem + kColdK, dka0 + uint64_t(((kk >> 2) * L::kSubBytes + (kk & 3) * 32) >> 4), dkb + uint64_t(kk * 128),
                            idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
                umma_commit(bar(kFBarQEmpty + st));
            }
            umma_commit(bar(kFBarFinal));
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
    if (warp == W_S) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace moda
