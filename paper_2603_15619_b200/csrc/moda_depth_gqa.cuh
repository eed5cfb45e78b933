// Depth part of the grouped-query forward as its own kernel (Sec. 3, "Group-aware depth KV calculation").
//
// At one position t the depth part is a small dense product with the G heads of a group as rows:
//     U = scale Q_t Kd_t^T   (G x l),      o_d = P Vd_t   (G x d),
// with Q_t the G query rows of the group at t and Kd_t, Vd_t the l depth rows of t (shared by the group).
// Warp-level MMAs (m16n8k16, heads as the 16-row operand) do both; a warp owns one position and walks the
// slots in groups with an online softmax.  The result is merged with what the sequence kernel, run
// without depth slots, left in O and LSE:
//     LSE = logaddexp(LSE_seq, LSE_dep),   O = w O_seq + (1 - w) O_dep,   w = exp(LSE_seq - LSE),
// which is the single softmax over the union of the two key sets.  The depth cache is read once per
// key/value head (not once per query head), in runs of kDgPos consecutive positions per 16-byte chunk.
#pragma once

#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "moda_cache.cuh"
#include "moda_decode.cuh"      // mma_bf16_16x8x16, ldmatrix_x4_trans
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kDgPos = 4;               // positions per CTA, one per warp: a 16-byte piece of 4 positions is a 64-byte run
constexpr int kDgThreads = kDgPos * 32;
constexpr int kDgRoundSlots = 16;        // slots staged per round
constexpr int kDgBufs = 2;              // rounds in flight: the next round's rows arrive while this round is used
template <int D> constexpr int dg_slots() { return kDgRoundSlots; }

struct DepthMergeParams {
    const __nv_bfloat16* Q;             // [B][T][H][d]
    const __nv_bfloat16* depth_kv;      // cache layout with Hk heads
    __nv_bfloat16* O;                   // in: sequence-only output; out: merged output
    float* LSE;                         // [B][H][T], likewise
    int B, T, H, Hk, l;
    int h0;                             // first head (inside its group of H / Hk) of the up to 8 heads this launch handles
    float scale_log2;
    int pm;                             // nonzero: depth_kv is in the position-major layout (moda_cache.cuh)
};

template <int D>
constexpr int depth_merge_smem_bytes() { return kDgBufs * 2 * kDgPos * dg_slots<D>() * D * 2; }

__device__ __forceinline__ void cp_async_16(uint32_t smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Byte offset of 16-byte piece `piece` of the row of (pos, slot) inside one staged tensor:
// rows of D bf16, pieces swizzled by the slot inside each 128-byte half so that the eight slots a
// fragment load touches fall into different banks.
template <int D>
__device__ __forceinline__ int dg_row_piece(int pos, int slot, int piece) {
    return ((pos * dg_slots<D>() + slot) * D * 2) + (((piece & 8) | ((piece & 7) ^ (slot & 7))) << 4);
}

template <int D, int G>
__global__ void __launch_bounds__(kDgThreads)
depth_merge_fwd_kernel(const DepthMergeParams p) {
    constexpr int CH = D / 8;                                  // 16-byte pieces per row
    constexpr int kDgSlots = dg_slots<D>();
    constexpr int kTensorBytes = kDgPos * kDgSlots * D * 2;    // staged K (then V) of one round
    extern __shared__ __align__(128) uint8_t dg_smem[];
    const int nblk = (p.T + kDgPos - 1) / kDgPos;
    const int blk = blockIdx.x % nblk;
    const int bh = blockIdx.x / nblk;
    const int hk = bh % p.Hk, b = bh / p.Hk;
    const int t0 = blk * kDgPos;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int t = t0 + warp;                                   // this warp's position
    const bool live = t < p.T;
    // More than 8 heads (G = 16): heads 8 .. 15 are rows 8 .. 15 of the same 16-row products, whose second half is
    // otherwise zero padding; a lane then carries the state of heads g and g + 8.
    constexpr bool kTwo = G > 8;

    // A fragments of Q_t: this lane's 8 features of head g for every 32 features (the same features it
    // takes from a depth key row below)
    uint4 qf[D / 32], qf2[kTwo ? D / 32 : 1];
#pragma unroll
    for (int kp = 0; kp < D / 32; ++kp) {
        qf[kp] = make_uint4(0u, 0u, 0u, 0u);
        if (live && g < G)
            qf[kp] = *reinterpret_cast<const uint4*>(p.Q + ((size_t(b) * p.T + t) * p.H + hk * (p.H / p.Hk) + p.h0 + g) * D + (4 * kp + tq) * 8);
        if constexpr (kTwo) {
            qf2[kp] = make_uint4(0u, 0u, 0u, 0u);
            if (live && g + 8 < G)
                qf2[kp] = *reinterpret_cast<const uint4*>(p.Q + ((size_t(b) * p.T + t) * p.H + hk * (p.H / p.Hk) + p.h0 + g + 8) * D + (4 * kp + tq) * 8);
        }
    }

    // the sequence kernel's output row and LSE of head g, requested now so that they are there at the end
    uint32_t os[D / 8];
    float lse_seq = 0.f;
    if (live && g < G) {
        const int h = hk * (p.H / p.Hk) + p.h0 + g;
        const __nv_bfloat16* orow = p.O + ((size_t(b) * p.T + t) * p.H + h) * D;
#pragma unroll
        for (int fb = 0; fb < D / 8; ++fb) os[fb] = *reinterpret_cast<const uint32_t*>(orow + 8 * fb + 2 * tq);
        lse_seq = p.LSE[(size_t(b) * p.H + h) * p.T + t];
    }
    uint32_t os2[kTwo ? D / 8 : 1];
    float lse_seq2 = 0.f;
    if constexpr (kTwo) {
        if (live && g + 8 < G) {
            const int h = hk * (p.H / p.Hk) + p.h0 + g + 8;
            const __nv_bfloat16* orow = p.O + ((size_t(b) * p.T + t) * p.H + h) * D;
#pragma unroll
            for (int fb = 0; fb < D / 8; ++fb) os2[fb] = *reinterpret_cast<const uint32_t*>(orow + 8 * fb + 2 * tq);
            lse_seq2 = p.LSE[(size_t(b) * p.H + h) * p.T + t];
        }
    }

    // cache addressing: block (slot, b, hk, tile, kv) holds [chunk][row 128][8]; the CTA's positions are rows
    // r0 .. r0 + kDgPos - 1 of tile t0 / 128 (kDgPos divides 128, so they never straddle tiles)
    const int tile = t0 / kTileRows, r0 = t0 % kTileRows;
    const size_t slot_elems = cache_slot_elems(p.B, p.T, p.Hk, D);
    const __nv_bfloat16* cbase = p.depth_kv + cache_block_offset(p.B, p.T, p.Hk, D, 0, b, hk, tile, 0) + size_t(r0) * 8;
    const uint32_t smem_base = smem_u32(dg_smem);

    float m_run = -INFINITY, lsum = 0.f;
    float m_run2 = -INFINITY, lsum2 = 0.f;                     // heads g + 8
    float o[D / 8][4];
#pragma unroll
    for (int fb = 0; fb < D / 8; ++fb) { o[fb][0] = 0.f; o[fb][1] = 0.f; o[fb][2] = 0.f; o[fb][3] = 0.f; }

    // stages the K and V rows of slots [s0, s0 + ns) of the CTA's positions into buffer `buf`: 16-byte pieces,
    // the positions of a piece are one contiguous run of the cache
    // A thread always copies the same (position, chunk) piece: kDgThreads is a multiple of kDgPos * CH, so only the
    // slot advances from one copy to the next.
    static_assert(kDgThreads % (kDgPos * CH) == 0, "one (position, chunk) per thread");
    constexpr int kSlotStep = kDgThreads / (kDgPos * CH);          // slots between a thread's copies
    const int st_pos = threadIdx.x % kDgPos, st_chunk = (threadIdx.x / kDgPos) % CH, st_slot0 = threadIdx.x / (kDgPos * CH);
    const __nv_bfloat16* st_src = cbase + (size_t(st_chunk) * kTileRows + st_pos) * 8;
    const uint32_t st_dst = smem_base + st_pos * kDgSlots * D * 2 + ((st_chunk & 8) << 4);
    // Position-major cache: a slot's K and V rows of the CTA's positions are one contiguous run of kDgPos * 4 d bytes;
    // consecutive threads copy consecutive 16-byte pieces of it (a warp request is 512 contiguous bytes).
    constexpr int kPmPieces = kDgPos * 2 * CH;                     // 16-byte pieces of that run
    static_assert(kDgThreads % kPmPieces == 0, "whole slots per pass");
    constexpr int kPmSlotStep = kDgThreads / kPmPieces;
    const int pm_q = threadIdx.x % kPmPieces, pm_slot0 = threadIdx.x / kPmPieces;
    const int pm_pos = pm_q / (2 * CH), pm_kv = (pm_q / CH) & 1, pm_chunk = pm_q % CH;
    const __nv_bfloat16* pm_src = p.depth_kv + cache_pm_offset(p.B, p.T, p.Hk, D, 0, b, hk, t0) + size_t(pm_q) * 8;
    const uint32_t pm_dst = smem_base + pm_kv * kTensorBytes + pm_pos * kDgSlots * D * 2 + ((pm_chunk & 8) << 4);
    auto stage_round = [&](int s0, int buf) {
        const int ns = min(kDgSlots, p.l - s0);
        if (p.pm) {
            const __nv_bfloat16* src = pm_src + size_t(s0 + pm_slot0) * slot_elems;
            const uint32_t dst = pm_dst + buf * 2 * kTensorBytes;
#pragma unroll
            for (int k = 0; k < kDgSlots / kPmSlotStep; ++k) {
                const int slot = pm_slot0 + k * kPmSlotStep;
                if (slot < ns)
                    cp_async_16(dst + slot * D * 2 + (((pm_chunk & 7) ^ (slot & 7)) << 4), src + size_t(k * kPmSlotStep) * slot_elems);
            }
            cp_async_commit();
            return;
        }
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            const __nv_bfloat16* src = st_src + size_t(s0 + st_slot0) * slot_elems + size_t(kv) * cache_block_elems(D);
            const uint32_t dst = st_dst + (buf * 2 + kv) * kTensorBytes;
#pragma unroll
            for (int k = 0; k < kDgSlots / kSlotStep; ++k) {
                const int slot = st_slot0 + k * kSlotStep;
                if (slot < ns)
                    cp_async_16(dst + slot * D * 2 + (((st_chunk & 7) ^ (slot & 7)) << 4), src + size_t(k * kSlotStep) * slot_elems);
            }
        }
        cp_async_commit();
    };
    if (p.l > 0) stage_round(0, 0);
#pragma unroll 1
    for (int s0 = 0, rnd = 0; s0 < p.l; s0 += kDgSlots, ++rnd) {
        const int ns = min(kDgSlots, p.l - s0);
        const int buf = rnd & 1;
        uint8_t* sK = dg_smem + (buf * 2) * kTensorBytes;
        uint8_t* sV = sK + kTensorBytes;
        // the other buffer was last read in round rnd - 1, which every warp has left (barrier below)
        if (s0 + kDgSlots < p.l) { stage_round(s0 + kDgSlots, buf ^ 1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        if (live) {
            // ---- scores of head g against 8 slots per block ----
            float sc[kDgSlots / 8][2], sc2[kDgSlots / 8][2];
#pragma unroll
            for (int nb = 0; nb < kDgSlots / 8; ++nb) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const int slot = 8 * nb + g;
                if (8 * nb < ns) {
#pragma unroll
                    for (int kp = 0; kp < D / 32; ++kp) {
                        const uint4 kvv = *reinterpret_cast<const uint4*>(sK + dg_row_piece<D>(warp, slot, 4 * kp + tq));
                        if constexpr (kTwo) {
                            mma_bf16_16x8x16(c, qf[kp].x, qf2[kp].x, qf[kp].y, qf2[kp].y, kvv.x, kvv.y);
                            mma_bf16_16x8x16(c, qf[kp].z, qf2[kp].z, qf[kp].w, qf2[kp].w, kvv.z, kvv.w);
                        } else {
                            mma_bf16_16x8x16(c, qf[kp].x, 0u, qf[kp].y, 0u, kvv.x, kvv.y);
                            mma_bf16_16x8x16(c, qf[kp].z, 0u, qf[kp].w, 0u, kvv.z, kvv.w);
                        }
                    }
                }
                sc[nb][0] = (8 * nb + 2 * tq < ns) ? c[0] * p.scale_log2 : -INFINITY;       // slots past l: stale rows
                sc[nb][1] = (8 * nb + 2 * tq + 1 < ns) ? c[1] * p.scale_log2 : -INFINITY;
                sc2[nb][0] = (8 * nb + 2 * tq < ns) ? c[2] * p.scale_log2 : -INFINITY;
                sc2[nb][1] = (8 * nb + 2 * tq + 1 < ns) ? c[3] * p.scale_log2 : -INFINITY;
            }
            float mx = -INFINITY;
#pragma unroll
            for (int nb = 0; nb < kDgSlots / 8; ++nb) mx = fmaxf(mx, fmaxf(sc[nb][0], sc[nb][1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run, mx);                  // finite: the round holds at least one slot
            const float alpha = fast_exp2(m_run - m_new);
            m_run = m_new;
            uint32_t pa[kDgSlots / 8];
            float psum = 0.f;
#pragma unroll
            for (int nb = 0; nb < kDgSlots / 8; ++nb) {
                const float p0 = fast_exp2(sc[nb][0] - m_new), p1 = fast_exp2(sc[nb][1] - m_new);
                psum += p0 + p1;
                pa[nb] = pack_bf16x2(p0, p1);
            }
            lsum = lsum * alpha + psum;
            if (alpha != 1.f) {
#pragma unroll
                for (int fb = 0; fb < D / 8; ++fb) { o[fb][0] *= alpha; o[fb][1] *= alpha; }
            }
            uint32_t pa2[kDgSlots / 8];
            if constexpr (kTwo) {                              // the same online-softmax step for head g + 8
                float mx2 = -INFINITY;
#pragma unroll
                for (int nb = 0; nb < kDgSlots / 8; ++nb) mx2 = fmaxf(mx2, fmaxf(sc2[nb][0], sc2[nb][1]));
                mx2 = fmaxf(mx2, __shfl_xor_sync(0xffffffffu, mx2, 1));
                mx2 = fmaxf(mx2, __shfl_xor_sync(0xffffffffu, mx2, 2));
                const float m_new2 = fmaxf(m_run2, mx2);
                const float alpha2 = fast_exp2(m_run2 - m_new2);
                m_run2 = m_new2;
                float psum2 = 0.f;
#pragma unroll
                for (int nb = 0; nb < kDgSlots / 8; ++nb) {
                    const float p0 = fast_exp2(sc2[nb][0] - m_new2), p1 = fast_exp2(sc2[nb][1] - m_new2);
                    psum2 += p0 + p1;
                    pa2[nb] = pack_bf16x2(p0, p1);
                }
                lsum2 = lsum2 * alpha2 + psum2;
                if (alpha2 != 1.f) {
#pragma unroll
                    for (int fb = 0; fb < D / 8; ++fb) { o[fb][2] *= alpha2; o[fb][3] *= alpha2; }
                }
            }
            // ---- o_d += P Vd: rows of slots past ns hold stale data with weight 0; zero them first if they
            //      could be NaN (they are rows of an earlier round or uninitialised shared memory) ----
            if (ns < kDgSlots) {
                for (int idx = lane; idx < (kDgSlots - ns) * CH; idx += 32) {
                    const int slot = ns + idx / CH, piece = idx % CH;
                    *reinterpret_cast<uint4*>(sV + dg_row_piece<D>(warp, slot, piece)) = make_uint4(0u, 0u, 0u, 0u);
                }
                __syncwarp();
            }
#pragma unroll
            for (int ks = 0; ks < kDgSlots / 16; ++ks) {
                if (16 * ks < ns) {
                    const int vslot = 16 * ks + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int fb = 0; fb < D / 8; fb += 2) {
                        const uint32_t addr = smem_u32(sV + dg_row_piece<D>(warp, vslot, fb + (lane >> 4)));
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                        if constexpr (kTwo) {
                            mma_bf16_16x8x16(o[fb], pa[2 * ks], pa2[2 * ks], pa[2 * ks + 1], pa2[2 * ks + 1], b0, b1);
                            mma_bf16_16x8x16(o[fb + 1], pa[2 * ks], pa2[2 * ks], pa[2 * ks + 1], pa2[2 * ks + 1], b2, b3);
                        } else {
                            mma_bf16_16x8x16(o[fb], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b0, b1);
                            mma_bf16_16x8x16(o[fb + 1], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b2, b3);
                        }
                    }
                }
            }
        }
        __syncthreads();                                       // this round's buffer may be refilled
    }

    // ---- merge with the sequence kernel's (O, LSE) of head g at position t ----
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    if (live && g < G) {
        const int h = hk * (p.H / p.Hk) + p.h0 + g;
        const float s2 = lse_seq * 1.4426950408889634f;            // sequence LSE in the log2 domain
        const float mt = fmaxf(s2, m_run);
        const float ws = fast_exp2(s2 - mt), wd = fast_exp2(m_run - mt);
        const float z = ws + wd * lsum;
        const float inv = 1.f / z;
        __nv_bfloat16* orow = p.O + ((size_t(b) * p.T + t) * p.H + h) * D;
#pragma unroll
        for (int fb = 0; fb < D / 8; ++fb) {
            const float a0 = (ws * bf16_lo_to_f32(os[fb]) + wd * o[fb][0]) * inv;
            const float a1 = (ws * bf16_hi_to_f32(os[fb]) + wd * o[fb][1]) * inv;
            *reinterpret_cast<uint32_t*>(orow + 8 * fb + 2 * tq) = pack_bf16x2(a0, a1);
        }
        if (tq == 0) p.LSE[(size_t(b) * p.H + h) * p.T + t] = (mt + log2f(z)) * 0.6931471805599453f;
    }
    if constexpr (kTwo) {
        lsum2 += __shfl_xor_sync(0xffffffffu, lsum2, 1);
        lsum2 += __shfl_xor_sync(0xffffffffu, lsum2, 2);
        if (live && g + 8 < G) {
            const int h = hk * (p.H / p.Hk) + p.h0 + g + 8;
            const float s2 = lse_seq2 * 1.4426950408889634f;
            const float mt = fmaxf(s2, m_run2);
            const float ws = fast_exp2(s2 - mt), wd = fast_exp2(m_run2 - mt);
            const float z = ws + wd * lsum2;
            const float inv = 1.f / z;
            __nv_bfloat16* orow = p.O + ((size_t(b) * p.T + t) * p.H + h) * D;
#pragma unroll
            for (int fb = 0; fb < D / 8; ++fb) {
                const float a0 = (ws * bf16_lo_to_f32(os2[fb]) + wd * o[fb][2]) * inv;
                const float a1 = (ws * bf16_hi_to_f32(os2[fb]) + wd * o[fb][3]) * inv;
                *reinterpret_cast<uint32_t*>(orow + 8 * fb + 2 * tq) = pack_bf16x2(a0, a1);
            }
            if (tq == 0) p.LSE[(size_t(b) * p.H + h) * p.T + t] = (mt + log2f(z)) * 0.6931471805599453f;
        }
    }
}


// =====================================================================================================
// Backward of the depth part for grouped-query calls, per position (derived from the forward above; the
// paper gives no backward).  With R = exp(U - LSE) (G x l; LSE is the forward's, over sequence and depth
// keys), D_g = <dO_g, O_g> and dU = R o (dO_t Vd_t^T - D):
//     dQ_t  += scale dU Kd_t          (G x d)
//     dKd_t  = scale dU^T Q_t         (l x d)   -- the contraction runs over the heads of the group, i.e. it
//     dVd_t  = R^T dO_t               (l x d)      is the sum over the group that the gradients need
// All five products are warp MMAs with the heads as the 16-row (or 16-deep) operand.  dU and R leave the
// first products in accumulator layout [head][slot]; the last two need them as [slot][head], which
// movmatrix provides (8 x 8 transposes across the warp).  Q_t and dO_t are also needed as B operands
// [head][feature]: they sit in shared memory and come through transposing matrix loads.
// The sequence kernel (run without depth slots) has left the sequence part of dQ; this kernel adds its share.
// =====================================================================================================
constexpr int kDbRoundSlots = 16;
template <int D> constexpr int db_pos() { return 256 / D; }           // positions per CTA (one per warp): 4 at d = 64, 2 at d = 128

struct DepthBwdParams {
    const __nv_bfloat16* Q;             // [B][T][H][d]
    const __nv_bfloat16* dO;
    const __nv_bfloat16* depth_kv;      // cache layout, Hk heads
    __nv_bfloat16* d_depth_kv;          // gradient cache, same layout
    __nv_bfloat16* dQ;                  // in: sequence part; out: sequence + depth part
    const float* LSE;                   // [B][H][T]
    const float* delta;                 // [B][H][T], D_t = <dO_t, O_t>
    int B, T, H, Hk, l;
    float scale, scale_log2;
    int accumulate;                     // depth gradients are added to d_depth_kv instead of stored
    int h0;                             // first head (inside its group of H / Hk) of the up to 8 heads this launch handles
    int pm;                             // nonzero: depth_kv and d_depth_kv are in the position-major layout (moda_cache.cuh)
};

template <int D, int G = 8>
struct DepthBwdSmem {
    static constexpr int P = db_pos<D>();
    static constexpr int kHeads = G > 8 ? 16 : 8;                       // head rows kept per position
    static constexpr int kIn = 2 * 2 * P * kDbRoundSlots * D * 2;       // two rounds x (K, V) rows
    static constexpr int kQd = kIn;                                     // Q_t and dO_t rows: [2][P][8 or 16 heads][D]
    static constexpr int kOut = kQd + 2 * P * kHeads * D * 2;           // dKd, dVd of the round: [2][P][16 slots][D]
    static constexpr int kTotal = kOut + 2 * P * kDbRoundSlots * D * 2;
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

template <int D, int G>
__global__ void __launch_bounds__(db_pos<D>() * 32, 4)
depth_bwd_gqa_kernel(const DepthBwdParams p) {
    using L = DepthBwdSmem<D, G>;
    constexpr bool kTwo = G > 8;                                   // heads 8 .. 15 as rows 8 .. 15 of the same products
    constexpr int HR = L::kHeads;
    constexpr int P = L::P, NT = P * 32, CH = D / 8, RS = kDbRoundSlots;
    constexpr int kTensorBytes = P * RS * D * 2;
    extern __shared__ __align__(128) uint8_t db_smem[];
    const uint32_t smem_base = smem_u32(db_smem);
    // byte offset of 16-byte piece `piece` of row `row` in a [rows][D] bf16 tile whose pieces are swizzled by the row
    auto row_piece = [](int row, int piece) { return row * D * 2 + (((piece & 8) | ((piece & 7) ^ (row & 7))) << 4); };

    const int nblk = num_tiles(p.T) * (kTileRows / P);             // whole tiles: the tail rows of the cache get zeros
    const int blk = blockIdx.x % nblk;
    const int bh = blockIdx.x / nblk;
    const int hk = bh % p.Hk, b = bh / p.Hk;
    const int t0 = blk * P;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int t = t0 + warp;
    const bool live = t < p.T;
    const bool head = live && g < G;
    const int h = hk * (p.H / p.Hk) + p.h0 + min(g, G - 1);
    const bool head2 = kTwo && live && g + 8 < G;
    const int h2 = hk * (p.H / p.Hk) + p.h0 + min(g + 8, G - 1);

    // ---- this position's Q and dO rows: A fragments in registers, and rows in shared memory for the B side ----
    uint4 qf[D / 32], gf[D / 32], qf2[kTwo ? D / 32 : 1], gf2[kTwo ? D / 32 : 1];
    uint8_t* sQ = db_smem + L::kQd + (0 * P + warp) * HR * D * 2;
    uint8_t* sG = db_smem + L::kQd + (1 * P + warp) * HR * D * 2;
#pragma unroll
    for (int kp = 0; kp < D / 32; ++kp) {
        qf[kp] = make_uint4(0u, 0u, 0u, 0u);
        gf[kp] = make_uint4(0u, 0u, 0u, 0u);
        if (head) {
            const size_t off = ((size_t(b) * p.T + t) * p.H + h) * D + (4 * kp + tq) * 8;
            qf[kp] = *reinterpret_cast<const uint4*>(p.Q + off);
            gf[kp] = *reinterpret_cast<const uint4*>(p.dO + off);
        }
        *reinterpret_cast<uint4*>(sQ + row_piece(g, 4 * kp + tq)) = qf[kp];       // rows of heads past G are zero
        *reinterpret_cast<uint4*>(sG + row_piece(g, 4 * kp + tq)) = gf[kp];
        if constexpr (kTwo) {
            qf2[kp] = make_uint4(0u, 0u, 0u, 0u);
            gf2[kp] = make_uint4(0u, 0u, 0u, 0u);
            if (head2) {
                const size_t off = ((size_t(b) * p.T + t) * p.H + h2) * D + (4 * kp + tq) * 8;
                qf2[kp] = *reinterpret_cast<const uint4*>(p.Q + off);
                gf2[kp] = *reinterpret_cast<const uint4*>(p.dO + off);
            }
            *reinterpret_cast<uint4*>(sQ + row_piece(g + 8, 4 * kp + tq)) = qf2[kp];
            *reinterpret_cast<uint4*>(sG + row_piece(g + 8, 4 * kp + tq)) = gf2[kp];
        }
    }
    float neg_lse2 = 0.f, dlt = 0.f, neg_lse2b = 0.f, dltb = 0.f;
    uint32_t dq_seq[D / 8], dq_seq2[kTwo ? D / 8 : 1];
    __nv_bfloat16* dq_row = p.dQ + ((size_t(b) * p.T + t) * p.H + h) * D;
    __nv_bfloat16* dq_row2 = p.dQ + ((size_t(b) * p.T + t) * p.H + h2) * D;
    if (head) {
        neg_lse2 = -p.LSE[(size_t(b) * p.H + h) * p.T + t] * 1.4426950408889634f;
        dlt = p.delta[(size_t(b) * p.H + h) * p.T + t];
#pragma unroll
        for (int fb = 0; fb < D / 8; ++fb) dq_seq[fb] = *reinterpret_cast<const uint32_t*>(dq_row + 8 * fb + 2 * tq);
    }
    if constexpr (kTwo) {
        if (head2) {
            neg_lse2b = -p.LSE[(size_t(b) * p.H + h2) * p.T + t] * 1.4426950408889634f;
            dltb = p.delta[(size_t(b) * p.H + h2) * p.T + t];
#pragma unroll
            for (int fb = 0; fb < D / 8; ++fb) dq_seq2[fb] = *reinterpret_cast<const uint32_t*>(dq_row2 + 8 * fb + 2 * tq);
        }
    }

    const int tile = t0 / kTileRows, r0 = t0 % kTileRows;
    const size_t slot_elems = cache_slot_elems(p.B, p.T, p.Hk, D);
    const size_t blk_off = cache_block_offset(p.B, p.T, p.Hk, D, 0, b, hk, tile, 0) + size_t(r0) * 8;
    const __nv_bfloat16* cbase = p.depth_kv + blk_off;
    __nv_bfloat16* gbase = p.d_depth_kv + blk_off;

    // a thread always moves the same (position, chunk) piece; only the slot advances
    static_assert(NT % (P * CH) == 0, "one (position, chunk) per thread");
    constexpr int kSlotStep = NT / (P * CH);
    const int st_pos = threadIdx.x % P, st_chunk = (threadIdx.x / P) % CH, st_slot0 = threadIdx.x / (P * CH);
    const size_t st_goff = (size_t(st_chunk) * kTileRows + st_pos) * 8;
    // Position-major layout: a slot's K and V rows of the CTA's positions are one run of P * 4 d bytes (see the forward)
    constexpr int kPmPieces = P * 2 * CH;
    static_assert(NT % kPmPieces == 0, "whole slots per pass");
    constexpr int kPmSlotStep = NT / kPmPieces;
    const int pm_q = threadIdx.x % kPmPieces, pm_slot0 = threadIdx.x / kPmPieces;
    const int pm_pos = pm_q / (2 * CH), pm_kv = (pm_q / CH) & 1, pm_chunk = pm_q % CH;
    const size_t pm_off = cache_pm_offset(p.B, p.T, p.Hk, D, 0, b, hk, t0) + size_t(pm_q) * 8;
    auto stage_round = [&](int s0, int buf) {
        const int ns = min(RS, p.l - s0);
        if (p.pm) {
            const __nv_bfloat16* src = p.depth_kv + pm_off + size_t(s0 + pm_slot0) * slot_elems;
            const uint32_t dst = smem_base + (buf * 2 + pm_kv) * kTensorBytes;
#pragma unroll
            for (int k = 0; k < RS / kPmSlotStep; ++k) {
                const int slot = pm_slot0 + k * kPmSlotStep;
                if (slot < ns) cp_async_16(dst + row_piece(pm_pos * RS + slot, pm_chunk), src + size_t(k * kPmSlotStep) * slot_elems);
            }
            cp_async_commit();
            return;
        }
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            const __nv_bfloat16* src = cbase + st_goff + size_t(s0 + st_slot0) * slot_elems + size_t(kv) * cache_block_elems(D);
            const uint32_t dst = smem_base + (buf * 2 + kv) * kTensorBytes;
#pragma unroll
            for (int k = 0; k < RS / kSlotStep; ++k) {
                const int slot = st_slot0 + k * kSlotStep;
                if (slot < ns) cp_async_16(dst + row_piece(st_pos * RS + slot, st_chunk), src + size_t(k * kSlotStep) * slot_elems);
            }
        }
        cp_async_commit();
    };

    float dq[D / 8][4];
#pragma unroll
    for (int fb = 0; fb < D / 8; ++fb) { dq[fb][0] = 0.f; dq[fb][1] = 0.f; dq[fb][2] = 0.f; dq[fb][3] = 0.f; }

    if (p.l > 0) stage_round(0, 0);
#pragma unroll 1
    for (int s0 = 0, rnd = 0; s0 < p.l; s0 += RS, ++rnd) {
        const int ns = min(RS, p.l - s0);
        const int buf = rnd & 1;
        const uint8_t* sK = db_smem + (buf * 2) * kTensorBytes + warp * RS * D * 2;     // this position's rows [slot][D]
        const uint8_t* sV = sK + kTensorBytes;
        uint8_t* oK = db_smem + L::kOut + (0 * P + warp) * RS * D * 2;                  // this position's output rows
        uint8_t* oV = db_smem + L::kOut + (1 * P + warp) * RS * D * 2;
        if (s0 + RS < p.l) { stage_round(s0 + RS, buf ^ 1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();                                   // the round's rows are in; the previous round's outputs are written out

        // ---- U = Q Kd^T and dO Vd^T for 16 slots (two blocks of 8) ----
        float cu[2][4], cv[2][4];
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { cu[nb][i] = 0.f; cv[nb][i] = 0.f; }
            const int slot = 8 * nb + g;
#pragma unroll
            for (int kp = 0; kp < D / 32; ++kp) {
                const uint4 kk = *reinterpret_cast<const uint4*>(sK + row_piece(slot, 4 * kp + tq));
                const uint4 vv = *reinterpret_cast<const uint4*>(sV + row_piece(slot, 4 * kp + tq));
                if constexpr (kTwo) {
                    mma_bf16_16x8x16(cu[nb], qf[kp].x, qf2[kp].x, qf[kp].y, qf2[kp].y, kk.x, kk.y);
                    mma_bf16_16x8x16(cu[nb], qf[kp].z, qf2[kp].z, qf[kp].w, qf2[kp].w, kk.z, kk.w);
                    mma_bf16_16x8x16(cv[nb], gf[kp].x, gf2[kp].x, gf[kp].y, gf2[kp].y, vv.x, vv.y);
                    mma_bf16_16x8x16(cv[nb], gf[kp].z, gf2[kp].z, gf[kp].w, gf2[kp].w, vv.z, vv.w);
                } else {
                    mma_bf16_16x8x16(cu[nb], qf[kp].x, 0u, qf[kp].y, 0u, kk.x, kk.y);
                    mma_bf16_16x8x16(cu[nb], qf[kp].z, 0u, qf[kp].w, 0u, kk.z, kk.w);
                    mma_bf16_16x8x16(cv[nb], gf[kp].x, 0u, gf[kp].y, 0u, vv.x, vv.y);
                    mma_bf16_16x8x16(cv[nb], gf[kp].z, 0u, gf[kp].w, 0u, vv.z, vv.w);
                }
            }
        }
        // ---- R and dU of head g for its slots 8 nb + 2 tq (+ 1); zero for slots past the end and heads past G,
        //      whose staged rows may hold anything ----
        uint32_t pr[2], pu[2], pr2[2] = {0u, 0u}, pu2[2] = {0u, 0u};
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
            float r[2], u[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const bool ok = head && (8 * nb + 2 * tq + e < ns);
                r[e] = ok ? fast_exp2(fmaf(cu[nb][e], p.scale_log2, neg_lse2)) : 0.f;
                u[e] = ok ? r[e] * (cv[nb][e] - dlt) : 0.f;
            }
            pr[nb] = pack_bf16x2(r[0], r[1]);
            pu[nb] = pack_bf16x2(u[0], u[1]);
            if constexpr (kTwo) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool ok = head2 && (8 * nb + 2 * tq + e < ns);
                    r[e] = ok ? fast_exp2(fmaf(cu[nb][2 + e], p.scale_log2, neg_lse2b)) : 0.f;
                    u[e] = ok ? r[e] * (cv[nb][2 + e] - dltb) : 0.f;
                }
                pr2[nb] = pack_bf16x2(r[0], r[1]);
                pu2[nb] = pack_bf16x2(u[0], u[1]);
            }
        }
        // ---- dQ share: dU (16 slots deep) x Kd rows; rows of slots past the end hold stale data: weight 0, but
        //      a NaN there would spread, so they are zeroed first ----
        if (ns < RS) {
            for (int idx = lane; idx < (RS - ns) * CH; idx += 32)
                *reinterpret_cast<uint4*>(const_cast<uint8_t*>(sK) + row_piece(ns + idx / CH, idx % CH)) = make_uint4(0u, 0u, 0u, 0u);
            __syncwarp();
        }
        {
            const int krow = ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
            for (int fb = 0; fb < D / 8; fb += 2) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(smem_u32(sK + row_piece(krow, fb + (lane >> 4))), b0, b1, b2, b3);
                mma_bf16_16x8x16(dq[fb], pu[0], pu2[0], pu[1], pu2[1], b0, b1);
                mma_bf16_16x8x16(dq[fb + 1], pu[0], pu2[0], pu[1], pu2[1], b2, b3);
            }
        }
        // ---- dKd = scale dU^T Q and dVd = R^T dO for the 16 slots: A = [slot][head] by 8 x 8 transposes ----
        {
            const uint32_t au0 = movmatrix_trans(pu[0]), au1 = movmatrix_trans(pu[1]);
            const uint32_t ar0 = movmatrix_trans(pr[0]), ar1 = movmatrix_trans(pr[1]);
            // heads 8 .. 15 are the second half of the contraction (k = 8 .. 15)
            uint32_t au2 = 0u, au3 = 0u, ar2 = 0u, ar3 = 0u;
            if constexpr (kTwo) {
                au2 = movmatrix_trans(pu2[0]); au3 = movmatrix_trans(pu2[1]);
                ar2 = movmatrix_trans(pr2[0]); ar3 = movmatrix_trans(pr2[1]);
            }
            const int hrow = lane & 7;                                  // head row a lane addresses for the matrix loads
#pragma unroll
            for (int fb = 0; fb < D / 8; fb += 4) {
                uint32_t q0, q1, q2, q3, g0, g1, g2, g3;                // B fragments [heads 0..7][8 features] of 4 blocks
                ldmatrix_x4_trans(smem_u32(sQ + row_piece(hrow, fb + (lane >> 3))), q0, q1, q2, q3);
                ldmatrix_x4_trans(smem_u32(sG + row_piece(hrow, fb + (lane >> 3))), g0, g1, g2, g3);
                const uint32_t qb[4] = {q0, q1, q2, q3}, gb[4] = {g0, g1, g2, g3};
                uint32_t qb2[4] = {0u, 0u, 0u, 0u}, gb2[4] = {0u, 0u, 0u, 0u};      // [heads 8..15][8 features]
                if constexpr (kTwo) {
                    ldmatrix_x4_trans(smem_u32(sQ + row_piece(hrow + 8, fb + (lane >> 3))), qb2[0], qb2[1], qb2[2], qb2[3]);
                    ldmatrix_x4_trans(smem_u32(sG + row_piece(hrow + 8, fb + (lane >> 3))), gb2[0], gb2[1], gb2[2], gb2[3]);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float ck[4] = {0.f, 0.f, 0.f, 0.f}, cw[4] = {0.f, 0.f, 0.f, 0.f};
                    mma_bf16_16x8x16(ck, au0, au1, au2, au3, qb[j], qb2[j]);
                    mma_bf16_16x8x16(cw, ar0, ar1, ar2, ar3, gb[j], gb2[j]);
                    // rows g (slot g) and g + 8, features 8 (fb + j) + 2 tq, + 1
                    const int piece = fb + j;
                    *reinterpret_cast<uint32_t*>(oK + row_piece(g, piece) + 4 * tq) = pack_bf16x2(ck[0] * p.scale, ck[1] * p.scale);
                    *reinterpret_cast<uint32_t*>(oK + row_piece(g + 8, piece) + 4 * tq) = pack_bf16x2(ck[2] * p.scale, ck[3] * p.scale);
                    *reinterpret_cast<uint32_t*>(oV + row_piece(g, piece) + 4 * tq) = pack_bf16x2(cw[0], cw[1]);
                    *reinterpret_cast<uint32_t*>(oV + row_piece(g + 8, piece) + 4 * tq) = pack_bf16x2(cw[2], cw[3]);
                }
            }
        }
        __syncthreads();                                   // all positions' output rows of this round are in shared memory
        // ---- write the round's gradients: a thread moves the (position, chunk) piece of every kSlotStep-th slot ----
        if (p.pm) {
            __nv_bfloat16* dst = p.d_depth_kv + pm_off + size_t(s0 + pm_slot0) * slot_elems;
            const uint8_t* src = db_smem + L::kOut + (pm_kv * P + pm_pos) * RS * D * 2;
#pragma unroll
            for (int k = 0; k < RS / kPmSlotStep; ++k) {
                const int slot = pm_slot0 + k * kPmSlotStep;
                if (slot < ns) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + row_piece(slot, pm_chunk));
                    __nv_bfloat16* out = dst + size_t(k * kPmSlotStep) * slot_elems;
                    if (p.accumulate) red_add_bf16x2_v4(out, v);
                    else *reinterpret_cast<uint4*>(out) = v;
                }
            }
        } else
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            __nv_bfloat16* dst = gbase + st_goff + size_t(s0 + st_slot0) * slot_elems + size_t(kv) * cache_block_elems(D);
            const uint8_t* src = db_smem + L::kOut + (kv * P + st_pos) * RS * D * 2;
#pragma unroll
            for (int k = 0; k < RS / kSlotStep; ++k) {
                const int slot = st_slot0 + k * kSlotStep;
                if (slot < ns) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + row_piece(slot, st_chunk));
                    __nv_bfloat16* out = dst + size_t(k * kSlotStep) * slot_elems;
                    if (p.accumulate) red_add_bf16x2_v4(out, v);
                    else *reinterpret_cast<uint4*>(out) = v;
                }
            }
        }
        // (the next round's barrier orders these reads before the next outputs)
    }

    // ---- dQ = sequence part + scale * depth part ----
    if (head) {
#pragma unroll
        for (int fb = 0; fb < D / 8; ++fb) {
            const float a0 = bf16_lo_to_f32(dq_seq[fb]) + p.scale * dq[fb][0];
            const float a1 = bf16_hi_to_f32(dq_seq[fb]) + p.scale * dq[fb][1];
            *reinterpret_cast<uint32_t*>(dq_row + 8 * fb + 2 * tq) = pack_bf16x2(a0, a1);
        }
    }
    if constexpr (kTwo) {
        if (head2) {
#pragma unroll
            for (int fb = 0; fb < D / 8; ++fb) {
                const float a0 = bf16_lo_to_f32(dq_seq2[fb]) + p.scale * dq[fb][2];
                const float a1 = bf16_hi_to_f32(dq_seq2[fb]) + p.scale * dq[fb][3];
                *reinterpret_cast<uint32_t*>(dq_row2 + 8 * fb + 2 * tq) = pack_bf16x2(a0, a1);
            }
        }
    }
}

}  // namespace moda
