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
// key/value head (not once per query head), in runs of kPos consecutive positions per 16-byte chunk.
#pragma once

#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "moda_cache.cuh"
#include "moda_decode.cuh"      // mma_bf16_16x8x16, ldmatrix_x4_trans
#include "sm100_ptx.cuh"

namespace moda {

constexpr int kDgPos = 8;               // positions per CTA, one per warp: a 16-byte piece of 8 positions is one 128-byte line
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
    float scale_log2;
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

    // A fragments of Q_t: this lane's 8 features of head g for every 32 features (the same features it
    // takes from a depth key row below)
    uint4 qf[D / 32];
#pragma unroll
    for (int kp = 0; kp < D / 32; ++kp) {
        qf[kp] = make_uint4(0u, 0u, 0u, 0u);
        if (live && g < G)
            qf[kp] = *reinterpret_cast<const uint4*>(p.Q + ((size_t(b) * p.T + t) * p.H + hk * G + g) * D + (4 * kp + tq) * 8);
    }

    // the sequence kernel's output row and LSE of head g, requested now so that they are there at the end
    uint32_t os[D / 8];
    float lse_seq = 0.f;
    if (live && g < G) {
        const int h = hk * G + g;
        const __nv_bfloat16* orow = p.O + ((size_t(b) * p.T + t) * p.H + h) * D;
#pragma unroll
        for (int fb = 0; fb < D / 8; ++fb) os[fb] = *reinterpret_cast<const uint32_t*>(orow + 8 * fb + 2 * tq);
        lse_seq = p.LSE[(size_t(b) * p.H + h) * p.T + t];
    }

    // cache addressing: block (slot, b, hk, tile, kv) holds [chunk][row 128][8]; the CTA's positions are rows
    // r0 .. r0 + kDgPos - 1 of tile t0 / 128 (kDgPos divides 128, so they never straddle tiles)
    const int tile = t0 / kTileRows, r0 = t0 % kTileRows;
    const size_t slot_elems = cache_slot_elems(p.B, p.T, p.Hk, D);
    const __nv_bfloat16* cbase = p.depth_kv + cache_block_offset(p.B, p.T, p.Hk, D, 0, b, hk, tile, 0) + size_t(r0) * 8;
    const uint32_t smem_base = smem_u32(dg_smem);

    float m_run = -INFINITY, lsum = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int fb = 0; fb < D / 8; ++fb) { o[fb][0] = 0.f; o[fb][1] = 0.f; o[fb][2] = 0.f; o[fb][3] = 0.f; }

    // stages the K and V rows of slots [s0, s0 + ns) of the CTA's positions into buffer `buf`: 16-byte pieces,
    // the eight positions of a piece are one 128-byte line of the cache
    // A thread always copies the same (position, chunk) piece: kDgThreads is a multiple of kDgPos * CH, so only the
    // slot advances from one copy to the next.
    static_assert(kDgThreads % (kDgPos * CH) == 0, "one (position, chunk) per thread");
    constexpr int kSlotStep = kDgThreads / (kDgPos * CH);          // slots between a thread's copies
    const int st_pos = threadIdx.x % kDgPos, st_chunk = (threadIdx.x / kDgPos) % CH, st_slot0 = threadIdx.x / (kDgPos * CH);
    const __nv_bfloat16* st_src = cbase + (size_t(st_chunk) * kTileRows + st_pos) * 8;
    const uint32_t st_dst = smem_base + st_pos * kDgSlots * D * 2 + ((st_chunk & 8) << 4);
    auto stage_round = [&](int s0, int buf) {
        const int ns = min(kDgSlots, p.l - s0);
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
            float sc[kDgSlots / 8][2];
#pragma unroll
            for (int nb = 0; nb < kDgSlots / 8; ++nb) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const int slot = 8 * nb + g;
                if (8 * nb < ns) {
#pragma unroll
                    for (int kp = 0; kp < D / 32; ++kp) {
                        const uint4 kvv = *reinterpret_cast<const uint4*>(sK + dg_row_piece<D>(warp, slot, 4 * kp + tq));
                        mma_bf16_16x8x16(c, qf[kp].x, 0u, qf[kp].y, 0u, kvv.x, kvv.y);
                        mma_bf16_16x8x16(c, qf[kp].z, 0u, qf[kp].w, 0u, kvv.z, kvv.w);
                    }
                }
                sc[nb][0] = (8 * nb + 2 * tq < ns) ? c[0] * p.scale_log2 : -INFINITY;       // slots past l: stale rows
                sc[nb][1] = (8 * nb + 2 * tq + 1 < ns) ? c[1] * p.scale_log2 : -INFINITY;
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
                        mma_bf16_16x8x16(o[fb], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b0, b1);
                        mma_bf16_16x8x16(o[fb + 1], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b2, b3);
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
        const int h = hk * G + g;
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
}

}  // namespace moda
