// Decode step of the MoDA operator (T_q = 1; paper Table 1, "decoding cache" / "decoding FLOPs"):
// the newest token of every sequence attends, under one softmax, to the T_kv keys of its layer's
// KV cache and to its own l depth key/value pairs (2 l H_k d values per token).
//
// The step reads every cached K and V row once and does 4 G d FLOPs per row, so it is bound by
// HBM; there is no contraction worth a tensor-core tile (G <= 8 query rows share a key).
//
//   decode_split_kernel   grid (split, kv head, batch): a CTA streams its share of the KV cache of
//                         one (b, kv head) once for all G query heads of the group.  Scores: one key
//                         per lane (the lane reads its key's row as 16-byte pieces and keeps it in
//                         registers; q sits in shared memory, pre-scaled, read as broadcasts), so no
//                         reduction across lanes.  Values: features across lanes (one coalesced row
//                         per load), the keys' weights broadcast through shared memory.  A warp has
//                         the 32 value rows of its pass and the 32 key rows of its next pass in
//                         flight at once (16 KiB at d = 128).  Each warp keeps an
//                         online-softmax state (m, l, o) per head; warps are merged through shared
//                         memory and the CTA writes one partial (m, l, o[d]) per head.
//   decode_merge_kernel   grid (query head, batch): merges the partials of all splits with the l
//                         depth pairs of the token (scored here: l d-length dot products) and writes
//                         O (bf16) and LSE (natural log).
#pragma once

#include <cstdint>
#include <cuda_bf16.h>
#include <cuda.h>
#include <cuda_runtime.h>

#include "sm100_ptx.cuh"

namespace moda {

constexpr int kDecodeWarps = 8;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kDecodeKeysPerPass = kDecodeWarps * 32;      // keys one CTA scores per pass
constexpr int kDecodeMaxSplits = 128;
constexpr float kDecodeLog2e = 1.4426950408889634f;
constexpr float kDecodeLn2 = 0.6931471805599453f;

struct DecodeParams {
    const __nv_bfloat16* q;       // [B][H][d]
    const __nv_bfloat16* K;       // [B][T_cap][Hk][d], rows [0, T_kv) valid
    const __nv_bfloat16* V;
    const __nv_bfloat16* depth;   // [l][B][Hk][2][d]: key row then value row of (slot, b, kv head)
    __nv_bfloat16* O;             // [B][H][d]
    float* LSE;                   // [B][H]
    float* part;                  // [B][Hk][S][G][d + 2]: m (log2 domain), l, o[d]
    int B, T_kv, T_cap, H, Hk, l;
    int S, keys_per_split;        // keys_per_split is a multiple of kDecodeKeysPerPass
    float scale_log2;             // scale * log2(e)
};

// Number of splits of the key range: enough CTAs for two to three waves of CTAs over the SMs, at
// least one pass of keys each.
inline int decode_num_splits(int B, int Hk, int T_kv, int num_sms) {
    const int passes = (T_kv + kDecodeKeysPerPass - 1) / kDecodeKeysPerPass;
    const int groups = B * Hk;
    int want = (4 * num_sms + groups - 1) / groups;
    if (want < 1) want = 1;
    if (want > passes) want = passes;
    if (want > kDecodeMaxSplits) want = kDecodeMaxSplits;
    return want;
}
inline int decode_keys_per_split(int T_kv, int S) {
    const int passes = (T_kv + kDecodeKeysPerPass - 1) / kDecodeKeysPerPass;
    return ((passes + S - 1) / S) * kDecodeKeysPerPass;
}
inline size_t decode_workspace_bytes(int B, int H, int d) {
    return size_t(B) * H * kDecodeMaxSplits * (d + 2) * 4;
}

// Shared-memory read that the compiler may not hoist out of the key loop: q is loop-invariant, and
// keeping G * d floats of it in registers spills.
__device__ __forceinline__ float4 lds_f32x4(const float* ptr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(ptr)))
                 : "memory");
    return v;
}

template <int D, int G>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_split_kernel(const DecodeParams p) {
    constexpr int CH = D / 8;                 // 16-byte pieces per row
    constexpr int FPL = D / 32;               // value features per lane (4 or 2)
    __shared__ __align__(16) float s_q[G * D];
    __shared__ float s_m[kDecodeWarps][G], s_l[kDecodeWarps][G];
    __shared__ __align__(16) float s_o[kDecodeWarps][G][D];
    __shared__ __align__(16) float s_p[kDecodeWarps][G][32];          // softmax weights of a warp's current pass

    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_begin = split * p.keys_per_split;
    const int k_end = min(p.T_kv, k_begin + p.keys_per_split);

    // q of the G heads of this group, scaled into the log2 domain
    for (int e = threadIdx.x; e < G * D; e += kDecodeThreads)
        s_q[e] = __bfloat162float(p.q[(size_t(b) * p.H + hk * G) * D + e]) * p.scale_log2;
    __syncthreads();

    const size_t row_stride = size_t(p.Hk) * D;                          // elements between positions
    const __nv_bfloat16* Kb = p.K + (size_t(b) * p.T_cap * p.Hk + hk) * D;
    const __nv_bfloat16* Vb = p.V + (size_t(b) * p.T_cap * p.Hk + hk) * D;

    float m[G], lsum[G], o[G][FPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY; lsum[g] = 0.f;
#pragma unroll
        for (int c = 0; c < FPL; ++c) o[g][c] = 0.f;
    }

    // The key rows of a pass sit in registers (one row per lane); they are dead once the scores are
    // formed, so the next pass's rows are requested right then and arrive during the softmax and the
    // value phase.  The 32 value rows of a pass are requested together (one coalesced row per load).
    uint4 kr[CH];
    auto load_keys = [&](int k0) {
        const int key = min(k0 + lane, k_end - 1);                        // lanes past the end repeat the last key
        const uint4* krow = reinterpret_cast<const uint4*>(Kb + size_t(key) * row_stride);
#pragma unroll
        for (int c = 0; c < CH; ++c) kr[c] = krow[c];
    };
    const int k_first = k_begin + warp * 32;
    if (k_first < k_end) load_keys(k_first);

#pragma unroll 1
    for (int k0 = k_first; k0 < k_end; k0 += kDecodeKeysPerPass) {
        const bool valid = k0 + lane < k_end;
        // ---- scores: this lane's key against the G heads; pieces outermost, heads inside, so that
        //      a piece's 8 unpacked values serve all G heads and die ----
        float sa[G], sb[G];
#pragma unroll
        for (int g = 0; g < G; ++g) { sa[g] = 0.f; sb[g] = 0.f; }
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const float k0f = bf16_lo_to_f32(kr[c].x), k1f = bf16_hi_to_f32(kr[c].x);
            const float k2f = bf16_lo_to_f32(kr[c].y), k3f = bf16_hi_to_f32(kr[c].y);
            const float k4f = bf16_lo_to_f32(kr[c].z), k5f = bf16_hi_to_f32(kr[c].z);
            const float k6f = bf16_lo_to_f32(kr[c].w), k7f = bf16_hi_to_f32(kr[c].w);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float4 qa = lds_f32x4(&s_q[g * D + 8 * c]);
                const float4 qb = lds_f32x4(&s_q[g * D + 8 * c + 4]);
                sa[g] = fmaf(qa.x, k0f, sa[g]); sb[g] = fmaf(qa.y, k1f, sb[g]);
                sa[g] = fmaf(qa.z, k2f, sa[g]); sb[g] = fmaf(qa.w, k3f, sb[g]);
                sa[g] = fmaf(qb.x, k4f, sa[g]); sb[g] = fmaf(qb.y, k5f, sb[g]);
                sa[g] = fmaf(qb.z, k6f, sa[g]); sb[g] = fmaf(qb.w, k7f, sb[g]);
            }
        }
        // ---- request this pass's value rows and the next pass's key rows ----
        const int n = min(32, k_end - k0);
        const __nv_bfloat16* vrow0 = Vb + size_t(k0) * row_stride + lane * FPL;
        uint32_t vr[32][FPL / 2];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const __nv_bfloat16* src = vrow0 + size_t(min(j, n - 1)) * row_stride;   // rows past the end repeat the last (weight 0)
            if constexpr (FPL == 4) {
                const uint2 v = *reinterpret_cast<const uint2*>(src);
                vr[j][0] = v.x; vr[j][1] = v.y;
            } else {
                vr[j][0] = *reinterpret_cast<const uint32_t*>(src);
            }
        }
        if (k0 + kDecodeKeysPerPass < k_end) load_keys(k0 + kDecodeKeysPerPass);
        // ---- online softmax over the 32 keys of this pass (the pass holds at least one key) ----
        __syncwarp();                                                     // the previous pass's weight reads are done
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float sg = valid ? sa[g] + sb[g] : -INFINITY;
            float mx = sg;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            const float m_new = fmaxf(m[g], mx);
            const float alpha = fast_exp2(m[g] - m_new);                 // 0 on the first pass
            const float pw = fast_exp2(sg - m_new);                      // 0 for lanes past the end
            s_p[warp][g][lane] = pw;
            lsum[g] = lsum[g] * alpha + pw;                              // per-lane share of the row sum
#pragma unroll
            for (int c = 0; c < FPL; ++c) o[g][c] *= alpha;
            m[g] = m_new;
        }
        __syncwarp();
        // ---- values: lanes across features; the weights of four keys come as one broadcast read ----
#pragma unroll
        for (int j4 = 0; j4 < 8; ++j4) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float4 w = lds_f32x4(&s_p[warp][g][4 * j4]);
                const float ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
                    for (int c = 0; c < FPL / 2; ++c) {
                        o[g][2 * c] = fmaf(ww[jj], bf16_lo_to_f32(vr[4 * j4 + jj][c]), o[g][2 * c]);
                        o[g][2 * c + 1] = fmaf(ww[jj], bf16_hi_to_f32(vr[4 * j4 + jj][c]), o[g][2 * c + 1]);
                    }
                }
            }
        }
    }

    // ---- merge the warps of this CTA ----
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float t = lsum[g];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
        if (lane == 0) { s_m[warp][g] = m[g]; s_l[warp][g] = t; }
#pragma unroll
        for (int c = 0; c < FPL; ++c) s_o[warp][g][lane * FPL + c] = o[g][c];
    }
    __syncthreads();
    float* out = p.part + ((size_t(b) * p.Hk + hk) * p.S + split) * G * (D + 2);
    for (int e = threadIdx.x; e < G * D; e += kDecodeThreads) {
        const int g = e / D, c = e - g * D;
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) mx = fmaxf(mx, s_m[w][g]);
        float acc = 0.f, lt = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float f = s_m[w][g] == -INFINITY ? 0.f : fast_exp2(s_m[w][g] - mx);   // a warp without keys
            acc = fmaf(f, s_o[w][g][c], acc);
            lt = fmaf(f, s_l[w][g], lt);
        }
        out[g * (D + 2) + 2 + c] = acc;
        if (c == 0) { out[g * (D + 2)] = mx; out[g * (D + 2) + 1] = lt; }
    }
}

// ---------------------------------------------------------------------------------------------
// The same split step with the KV cache staged through shared memory by TMA.  A producer warp keeps a
// ring of stages (64 keys: their K rows and V rows as 128-byte-swizzled boxes) in flight, 128 KiB
// per SM, more than HBM latency times the SM's share of bandwidth; consumer warp pair p handles stages
// p, p + 4, ... (32 keys per warp), always in the same ring slots.  The arithmetic is that of decode_split_kernel: one key per lane
// for the scores, lanes across features for the values.
// ---------------------------------------------------------------------------------------------
constexpr int kDecodeStageKeys = 64;
constexpr int kDecodeConsumerWarps = 8;
constexpr int kDecodeTmaThreads = (kDecodeConsumerWarps + 1) * 32;
constexpr int kDecodePairs = kDecodeConsumerWarps / 2;

template <int D, int G>
struct DecodeSmem {
    static constexpr int kStageBytes = 2 * kDecodeStageKeys * D * 2;           // K box(es) + V box(es)
    static constexpr int kFixed = G * D * 4 + kDecodeConsumerWarps * G * 32 * 4 + 2 * kDecodeConsumerWarps * G * 4 + 256;
    static constexpr int kMergeBytes = kDecodeConsumerWarps * G * D * 4;      // aliases the ring at the end
    static constexpr int kAvail = 227 * 1024 - 1024 - kFixed;
    static constexpr int kStagesFit = kAvail / kStageBytes;
    // A multiple of the number of consumer pairs, so that a ring slot is always read by the same pair.
    // (mbarrier waits tell phases apart by one parity bit: a waiter may be at most one phase ahead of
    // its barrier, which holds when the slot's uses are consumed in order by the same warps, and does
    // not when pairs alternate on a slot and one of them runs ahead.)
    static constexpr int kStages = kStagesFit >= 2 * kDecodePairs ? 2 * kDecodePairs : kDecodePairs;
    static constexpr int kRing = 0;
    static constexpr int kQ = kStages * kStageBytes;
    static constexpr int kP = kQ + G * D * 4;
    static constexpr int kM = kP + kDecodeConsumerWarps * G * 32 * 4;
    static constexpr int kL = kM + kDecodeConsumerWarps * G * 4;
    static constexpr int kBars = kL + kDecodeConsumerWarps * G * 4;           // full[kStages], empty[kStages], abort word
    static constexpr int kDynamic = kBars + 2 * 8 * 8 + 16 + 1024;            // + alignment slack
    static_assert(kStagesFit >= kDecodePairs && kStages % kDecodePairs == 0, "ring too small");
    static_assert(kMergeBytes <= kStages * kStageBytes, "merge buffer must fit in the ring");
};

template <int D, int G>
__global__ void __launch_bounds__(kDecodeTmaThreads, 1)
decode_split_tma_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                        const DecodeParams p) {
    using L = DecodeSmem<D, G>;
    constexpr int CH = D / 8, FPL = D / 32, NH = D / 64;                     // NH 64-feature boxes per row
    constexpr int kBoxBytes = kDecodeStageKeys * 128;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* s_q = reinterpret_cast<float*>(smem + L::kQ);
    float* s_p = reinterpret_cast<float*>(smem + L::kP);
    float* s_m = reinterpret_cast<float*>(smem + L::kM);
    float* s_l = reinterpret_cast<float*>(smem + L::kL);
    const uint32_t bars = smem_u32(smem + L::kBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kBars + 2 * 8 * 8);
    auto full_bar = [&](int st) { return bars + st * 8; };
    auto empty_bar = [&](int st) { return bars + (8 + st) * 8; };

    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_begin = split * p.keys_per_split;
    const int k_end = min(p.T_kv, k_begin + p.keys_per_split);
    const int n_stage = (k_end - k_begin + kDecodeStageKeys - 1) / kDecodeStageKeys;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int st = 0; st < L::kStages; ++st) { mbar_init(full_bar(st), 1); mbar_init(empty_bar(st), 2); }
        fence_mbar_init();
    }
    for (int e = threadIdx.x; e < G * D; e += kDecodeTmaThreads)
        s_q[e] = __bfloat162float(p.q[(size_t(b) * p.H + hk * G) * D + e]) * p.scale_log2;
    __syncthreads();

    float m[G], lsum[G], o[G][FPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY; lsum[g] = 0.f;
#pragma unroll
        for (int c = 0; c < FPL; ++c) o[g][c] = 0.f;
    }

    int n_issued = 0;                                                   // producer lane: stages requested so far
    if (warp == kDecodeConsumerWarps) {
        // ---- producer: one lane keeps the ring full ----
        if (lane == 0) {
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            for (int i = 0; i < n_stage; ++i) {
                const int st = i % L::kStages;
                if (i >= L::kStages) mbar_wait(empty_bar(st), ((i / L::kStages) - 1) & 1, abort_flag, 70);
                if (*abort_flag != 0) break;
                const uint32_t dst = smem_u32(smem + L::kRing + st * L::kStageBytes);
                mbar_arrive_expect_tx(full_bar(st), L::kStageBytes);
                const int t0 = k_begin + i * kDecodeStageKeys;
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    tma_load_4d(dst + h * kBoxBytes, &mapK, full_bar(st), 64 * h, hk, t0, b);
                    tma_load_4d(dst + (NH + h) * kBoxBytes, &mapV, full_bar(st), 64 * h, hk, t0, b);
                }
                n_issued = i + 1;
            }
        }
    } else {
        // ---- consumers: warp pair `pair` takes stages pair, pair + 4, ...; this warp its `half` of 32 keys ----
        const int pair = warp >> 1, half = warp & 1;
        float* my_p = s_p + warp * G * 32;
#pragma unroll 1
        for (int i = pair; i < n_stage; i += kDecodePairs) {
            const int st = i % L::kStages;
            mbar_wait(full_bar(st), (i / L::kStages) & 1, abort_flag, 71);
            if (__shfl_sync(0xffffffffu, *abort_flag, 0) != 0) break;      // one lane's view, so the warp leaves together
            const int k0 = k_begin + i * kDecodeStageKeys + half * 32;     // first key of this warp
            const int n = min(32, k_end - k0);                             // may be <= 0 for the second half of the last stage
            if (n > 0) {
                const uint8_t* sK = smem + L::kRing + st * L::kStageBytes;
                const uint8_t* sV = sK + NH * kBoxBytes;
                const int r = half * 32 + lane;                            // row of this lane's key in the stage
                const bool valid = lane < n;
                float sa[G], sb[G];
#pragma unroll
                for (int g = 0; g < G; ++g) { sa[g] = 0.f; sb[g] = 0.f; }
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const uint4 kv = *reinterpret_cast<const uint4*>(sK + (c >> 3) * kBoxBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4));
                    const float k0f = bf16_lo_to_f32(kv.x), k1f = bf16_hi_to_f32(kv.x);
                    const float k2f = bf16_lo_to_f32(kv.y), k3f = bf16_hi_to_f32(kv.y);
                    const float k4f = bf16_lo_to_f32(kv.z), k5f = bf16_hi_to_f32(kv.z);
                    const float k6f = bf16_lo_to_f32(kv.w), k7f = bf16_hi_to_f32(kv.w);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float4 qa = lds_f32x4(&s_q[g * D + 8 * c]);
                        const float4 qb = lds_f32x4(&s_q[g * D + 8 * c + 4]);
                        sa[g] = fmaf(qa.x, k0f, sa[g]); sb[g] = fmaf(qa.y, k1f, sb[g]);
                        sa[g] = fmaf(qa.z, k2f, sa[g]); sb[g] = fmaf(qa.w, k3f, sb[g]);
                        sa[g] = fmaf(qb.x, k4f, sa[g]); sb[g] = fmaf(qb.y, k5f, sb[g]);
                        sa[g] = fmaf(qb.z, k6f, sa[g]); sb[g] = fmaf(qb.w, k7f, sb[g]);
                    }
                }
                __syncwarp();                                              // the previous stage's weight reads are done
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float sg = valid ? sa[g] + sb[g] : -INFINITY;    // rows past T_kv may hold anything
                    float mx = sg;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                    const float m_new = fmaxf(m[g], mx);
                    const float alpha = fast_exp2(m[g] - m_new);
                    const float pw = fast_exp2(sg - m_new);
                    my_p[g * 32 + lane] = pw;
                    lsum[g] = lsum[g] * alpha + pw;
#pragma unroll
                    for (int c = 0; c < FPL; ++c) o[g][c] *= alpha;
                    m[g] = m_new;
                }
                __syncwarp();
                // values: this lane's FPL features of every row; rows past the end repeat the last one (weight 0)
                const int vbox = (lane * FPL) >> 6;                        // which 64-feature box
                const int vchunk = ((lane * FPL) & 63) >> 3;               // 16-byte piece inside the 128-byte row
                const int vsub = ((lane * FPL) & 7) * 2;                   // byte offset inside the piece
#pragma unroll
                for (int j4 = 0; j4 < 8; ++j4) {
                    uint32_t vr[4][FPL / 2];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const int rr = half * 32 + min(4 * j4 + jj, n - 1);
                        const uint8_t* src = sV + vbox * kBoxBytes + rr * 128 + ((vchunk ^ (rr & 7)) << 4) + vsub;
                        if constexpr (FPL == 4) {
                            const uint2 v = *reinterpret_cast<const uint2*>(src);
                            vr[jj][0] = v.x; vr[jj][1] = v.y;
                        } else {
                            vr[jj][0] = *reinterpret_cast<const uint32_t*>(src);
                        }
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float4 w = lds_f32x4(&my_p[g * 32 + 4 * j4]);
                        const float ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
                            for (int c = 0; c < FPL / 2; ++c) {
                                o[g][2 * c] = fmaf(ww[jj], bf16_lo_to_f32(vr[jj][c]), o[g][2 * c]);
                                o[g][2 * c + 1] = fmaf(ww[jj], bf16_hi_to_f32(vr[jj][c]), o[g][2 * c + 1]);
                            }
                        }
                    }
                }
            }
            // the stage is refilled by the async proxy: order this warp's reads before the arrival
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(st));
        }
    }

    // ---- merge the consumer warps (the ring is idle now: its memory holds the per-warp outputs) ----
    __syncthreads();
    if (*abort_flag != 0) {
        // a wait gave up: the copies requested last may still be in flight; let them land (bounded
        // wait on the latest use of each slot) before the CTA's shared memory is released
        if (threadIdx.x == kDecodeConsumerWarps * 32) {
            for (int i = max(0, n_issued - L::kStages); i < n_issued; ++i)
                for (int spin = 0; spin < (1 << 20); ++spin)
                    if (mbar_try_wait(full_bar(i % L::kStages), (i / L::kStages) & 1)) break;
        }
        return;
    }
    float* s_o = reinterpret_cast<float*>(smem + L::kRing);
    if (warp < kDecodeConsumerWarps) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float t = lsum[g];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
            if (lane == 0) { s_m[warp * G + g] = m[g]; s_l[warp * G + g] = t; }
#pragma unroll
            for (int c = 0; c < FPL; ++c) s_o[(warp * G + g) * D + lane * FPL + c] = o[g][c];
        }
    }
    __syncthreads();
    float* out = p.part + ((size_t(b) * p.Hk + hk) * p.S + split) * G * (D + 2);
    for (int e = threadIdx.x; e < G * D; e += kDecodeTmaThreads) {
        const int g = e / D, c = e - g * D;
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeConsumerWarps; ++w) mx = fmaxf(mx, s_m[w * G + g]);
        float acc = 0.f, lt = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeConsumerWarps; ++w) {
            const float f = s_m[w * G + g] == -INFINITY ? 0.f : fast_exp2(s_m[w * G + g] - mx);   // a warp without keys
            acc = fmaf(f, s_o[(w * G + g) * D + c], acc);
            lt = fmaf(f, s_l[w * G + g], lt);
        }
        out[g * (D + 2) + 2 + c] = acc;
        if (c == 0) { out[g * (D + 2)] = mx; out[g * (D + 2) + 1] = lt; }
    }
}

// One CTA of D threads per (b, query head): thread = output feature.
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const DecodeParams p) {
    __shared__ float s_w[kDecodeMaxSplits];          // weight of each split's partial
    __shared__ float s_d[256];                       // depth scores (log2 domain), then weights; l <= 256
    __shared__ float s_q[D];
    __shared__ float s_red[D / 32];
    const int h = blockIdx.x, b = blockIdx.y;
    const int G = p.H / p.Hk, hk = h / G, g = h - hk * G;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int NW = D / 32;

    s_q[tid] = __bfloat162float(p.q[(size_t(b) * p.H + h) * D + tid]) * p.scale_log2;
    __syncthreads();
    // depth scores: one warp per slot, lanes across features
    for (int i = warp; i < p.l; i += NW) {
        const __nv_bfloat16* kd = p.depth + ((size_t(i) * p.B + b) * p.Hk + hk) * 2 * D;
        float a = 0.f;
#pragma unroll
        for (int c = lane; c < D; c += 32) a = fmaf(s_q[c], __bfloat162float(kd[c]), a);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        if (lane == 0) s_d[i] = a;
    }
    __syncthreads();
    const float* part = p.part + ((size_t(b) * p.Hk + hk) * p.S * G + g) * (D + 2);   // + split * G * (D + 2)
    const size_t split_stride = size_t(G) * (D + 2);
    // global maximum over the split maxima and the depth scores
    float mx = -INFINITY;
    for (int s = tid; s < p.S; s += D) mx = fmaxf(mx, part[s * split_stride]);
    for (int i = tid; i < p.l; i += D) mx = fmaxf(mx, s_d[i]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = s_red[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) mx = fmaxf(mx, s_red[w]);
    __syncthreads();
    // weights and the row sum
    float lt = 0.f;
    for (int s = tid; s < p.S; s += D) {
        const float ms = part[s * split_stride];
        const float f = ms == -INFINITY ? 0.f : fast_exp2(ms - mx);
        s_w[s] = f;
        lt = fmaf(f, part[s * split_stride + 1], lt);
    }
    for (int i = tid; i < p.l; i += D) {
        const float w = fast_exp2(s_d[i] - mx);
        s_d[i] = w;
        lt += w;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) lt += __shfl_xor_sync(0xffffffffu, lt, off);
    if (lane == 0) s_red[warp] = lt;
    __syncthreads();
    lt = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) lt += s_red[w];
    // output feature tid
    float acc = 0.f;
    for (int s = 0; s < p.S; ++s) acc = fmaf(s_w[s], part[s * split_stride + 2 + tid], acc);
    for (int i = 0; i < p.l; ++i) {
        const __nv_bfloat16* vd = p.depth + (((size_t(i) * p.B + b) * p.Hk + hk) * 2 + 1) * D;
        acc = fmaf(s_d[i], __bfloat162float(vd[tid]), acc);
    }
    p.O[(size_t(b) * p.H + h) * D + tid] = __float2bfloat16(acc / lt);
    if (tid == 0) p.LSE[size_t(b) * p.H + h] = (mx + log2f(lt)) * kDecodeLn2;
}

}  // namespace moda
