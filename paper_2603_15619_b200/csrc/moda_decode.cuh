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
//                         per load), the key's weight broadcast with a shuffle.  Each warp keeps an
//                         online-softmax state (m, l, o) per head; warps are merged through shared
//                         memory and the CTA writes one partial (m, l, o[d]) per head.
//   decode_merge_kernel   grid (query head, batch): merges the partials of all splits with the l
//                         depth pairs of the token (scored here: l d-length dot products) and writes
//                         O (bf16) and LSE (natural log).
#pragma once

#include <cstdint>
#include <cuda_bf16.h>
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
                 : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(ptr))));
    return v;
}

template <int D, int G>
__global__ void __launch_bounds__(kDecodeThreads, G <= 4 ? 2 : 1)
decode_split_kernel(const DecodeParams p) {
    constexpr int CH = D / 8;                 // 16-byte pieces per row
    constexpr int FPL = D / 32;               // value features per lane (4 or 2)
    __shared__ __align__(16) float s_q[G * D];
    __shared__ float s_m[kDecodeWarps][G], s_l[kDecodeWarps][G];
    __shared__ __align__(16) float s_o[kDecodeWarps][G][D];

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

#pragma unroll 1
    for (int k0 = k_begin + warp * 32; k0 < k_end; k0 += kDecodeKeysPerPass) {
        const int key = k0 + lane;
        const bool valid = key < k_end;
        // ---- scores: this lane's key against the G heads ----
        uint4 kr[CH];
        const uint4* krow = reinterpret_cast<const uint4*>(Kb + size_t(valid ? key : k0) * row_stride);
#pragma unroll
        for (int c = 0; c < CH; ++c) kr[c] = krow[c];
        // pieces outermost, heads inside: a piece's 8 unpacked values serve all G heads and die
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
        float s[G];
#pragma unroll
        for (int g = 0; g < G; ++g) s[g] = valid ? sa[g] + sb[g] : -INFINITY;
        // ---- online softmax over the 32 keys of this pass (the pass holds at least one key) ----
        float pw[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float mx = s[g];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            const float m_new = fmaxf(m[g], mx);
            const float alpha = fast_exp2(m[g] - m_new);                 // 0 on the first pass
            pw[g] = fast_exp2(s[g] - m_new);                             // 0 for lanes past the end
            lsum[g] = lsum[g] * alpha + pw[g];                           // per-lane share of the row sum
#pragma unroll
            for (int c = 0; c < FPL; ++c) o[g][c] *= alpha;
            m[g] = m_new;
        }
        // ---- values: lanes across features, one coalesced row per load, weights by shuffle ----
        const int n = min(32, k_end - k0);
        const __nv_bfloat16* vrow0 = Vb + size_t(k0) * row_stride + lane * FPL;
#pragma unroll 1
        for (int j0 = 0; j0 < n; j0 += 8) {
            uint32_t vr[8][FPL / 2];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int jj = min(j0 + j, n - 1);                        // rows past the end repeat the last one (weight 0)
                const __nv_bfloat16* src = vrow0 + size_t(jj) * row_stride;
                if constexpr (FPL == 4) {
                    const uint2 v = *reinterpret_cast<const uint2*>(src);
                    vr[j][0] = v.x; vr[j][1] = v.y;
                } else {
                    vr[j][0] = *reinterpret_cast<const uint32_t*>(src);
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float w = __shfl_sync(0xffffffffu, pw[g], j0 + j);     // lanes >= n hold 0
#pragma unroll
                    for (int c = 0; c < FPL / 2; ++c) {
                        o[g][2 * c] = fmaf(w, bf16_lo_to_f32(vr[j][c]), o[g][2 * c]);
                        o[g][2 * c + 1] = fmaf(w, bf16_hi_to_f32(vr[j][c]), o[g][2 * c + 1]);
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
