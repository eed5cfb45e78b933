// Decode step of the MoDA operator (T_q = 1; paper Table 1, "decoding cache" / "decoding FLOPs"):
// the newest token of every sequence attends, under one softmax, to the T_kv keys of its layer's
// KV cache and to its own l depth key/value pairs (2 l H_k d values per token).
//
// The step reads every cached K and V row once and does 4 G d FLOPs per row, so it is bound by
// HBM; G <= 8 query rows share a key, too few for a tcgen05 tile (64 or 128 rows).
//
//   decode_split_tma_kernel  persistent, one CTA per SM, over work items (batch, kv head, split of the key
//                         range).  A producer lane keeps a ring of TMA stages (64 keys: their K rows and V
//                         rows as 128-byte-swizzled boxes) in flight, 128 KiB per SM, and runs ahead into
//                         the CTA's next work item, so the HBM stream does not stop at item boundaries.
//                         Eight consumer warps, 32 keys of a stage each: scores and weighted values with
//                         warp-level MMAs whose 16-row operand holds the G <= 8 heads of the group (the
//                         CUDA-core form of the same arithmetic is issue-bound from G = 4 on); K pieces
//                         and, through transposing matrix loads, V pieces come from the swizzled stage.
//                         Each warp keeps an online-softmax state (m, l, o) per head; at the end of an
//                         item the warps are merged through shared memory and the CTA writes one partial
//                         (m, l, o[d]) per head.
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
    int num_sms;
    int kv_rep;                   // groups of more than 8 query heads run as kv_rep groups of 8 on the same K, V head
    const int* seq_lens;          // [B] cached positions per sequence (each 1 .. T_kv), or null: T_kv for all
    const int* block_table;       // paged cache: [B][max_blocks] page of every block of page_size positions, or null
    int page_size, max_blocks;    // paged cache: K, V are [num_pages][page_size][Hk][d]; page_size is a multiple of 64
    float scale_log2;             // scale * log2(e)
};

// Split of the key range of every (batch, kv head) group into S work items of `passes_per_split`
// passes (256 keys) each.  The persistent CTAs take items round-robin, so the step lasts as long as the
// CTA with the most work: ceil(items / SMs) items of passes_per_split passes plus a fixed cost per item
// (merge, partial write; about a third of a pass).  The plan with the smallest such estimate wins.
struct DecodePlan { int S, keys_per_split; };
inline DecodePlan decode_plan(int B, int Hk, int T_kv, int num_sms) {
    const int passes = (T_kv + kDecodeKeysPerPass - 1) / kDecodeKeysPerPass;
    const long long groups = (long long)B * Hk;
    DecodePlan best{1, passes * kDecodeKeysPerPass};
    double best_cost = 1e300;
    for (int pp = passes; pp >= 1; --pp) {
        const int S = (passes + pp - 1) / pp;
        if (S > kDecodeMaxSplits) break;
        const long long items = groups * S;
        const long long rounds = (items + num_sms - 1) / num_sms;
        const double cost = double(rounds) * (pp + 0.35);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = DecodePlan{S, pp * kDecodeKeysPerPass}; }
    }
    return best;
}
inline size_t decode_workspace_bytes(int B, int H, int d) {
    return size_t(B) * H * kDecodeMaxSplits * (d + 2) * 4;
}

// Warp-level tensor-core primitives (bf16 inputs, fp32 accumulate).  The decode step is bound by HBM and
// its contraction has at most 8 rows, far below the 64 / 128 rows of a tcgen05 tile.
__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t smem_addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(smem_addr) : "memory");
}

constexpr int kDecodeStageKeys = 64;
constexpr int kDecodeConsumerWarps = 8;
constexpr int kDecodeConsumerThreads = kDecodeConsumerWarps * 32;
constexpr int kDecodeTmaThreads = kDecodeConsumerThreads + 32;
constexpr int kDecodePairs = kDecodeConsumerWarps / 2;

template <int D, int G>
struct DecodeSmem {
    static constexpr int kStageBytes = 2 * kDecodeStageKeys * D * 2;           // K box(es) + V box(es)
    // A multiple of the number of consumer pairs, so that a ring slot is always read by the same pair.
    // (mbarrier waits tell phases apart by one parity bit: a waiter may be at most one phase ahead of
    // its barrier, which holds when the slot's uses are consumed in order by the same warps, and does
    // not when pairs alternate on a slot and one of them runs ahead.)
    static constexpr int kStages = (D == 64 ? 2 : 1) * kDecodePairs;           // 128 KiB in flight
    static constexpr int kRing = 0;
    static constexpr int kQ = kStages * kStageBytes;                           // two buffers of 8 bf16 rows: this item's q, the next one's
    static constexpr int kO = kQ + 2 * 8 * D * 2;                              // per-warp outputs for the merge
    static constexpr int kM = kO + kDecodeConsumerWarps * G * D * 4;
    static constexpr int kL = kM + kDecodeConsumerWarps * G * 4;
    static constexpr int kBars = kL + kDecodeConsumerWarps * G * 4;           // full[8], empty[8], abort word
    static constexpr int kDynamic = kBars + 2 * 8 * 8 + 16 + 1024;            // + alignment slack
    static_assert(kStages <= 8 && kStages % kDecodePairs == 0, "ring slots must map to fixed pairs");
    static_assert(kDynamic <= 227 * 1024, "shared memory");
};

__device__ __forceinline__ void decode_consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kDecodeConsumerThreads) : "memory");
}

template <int D, int G>
__global__ void __launch_bounds__(kDecodeTmaThreads, 1)
decode_split_tma_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                        const DecodeParams p) {
    using L = DecodeSmem<D, G>;
    constexpr int CH = D / 8, NH = D / 64;                                    // NH 64-feature boxes per row
    constexpr int kBoxBytes = kDecodeStageKeys * 128;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint4* s_qbuf = reinterpret_cast<uint4*>(smem + L::kQ);
    float* s_o = reinterpret_cast<float*>(smem + L::kO);
    float* s_m = reinterpret_cast<float*>(smem + L::kM);
    float* s_l = reinterpret_cast<float*>(smem + L::kL);
    const uint32_t bars = smem_u32(smem + L::kBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kBars + 2 * 8 * 8);
    auto full_bar = [&](int st) { return bars + st * 8; };
    auto empty_bar = [&](int st) { return bars + (8 + st) * 8; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_items = p.B * p.Hk * p.S;
    // work item -> (batch, kv head, split) and its key range
    struct Item { int b, hk, split, k_begin, k_end, n_stage; };
    auto item_of = [&](int it) {
        Item w;
        // split-major order: a CTA's items (it, it + grid, ...) then come from all parts of the key range, so
        // the empty late splits of short sequences spread over the CTAs instead of emptying some of them
        const int groups = p.B * p.Hk;
        w.split = it / groups;
        const int bh = it - w.split * groups;
        w.hk = bh % p.Hk;
        w.b = bh / p.Hk;
        w.k_begin = w.split * p.keys_per_split;
        const int len = p.seq_lens ? min(max(p.seq_lens[w.b], 1), p.T_kv) : p.T_kv;   // this sequence's cached positions
        w.k_end = min(len, w.k_begin + p.keys_per_split);
        w.n_stage = max(0, (w.k_end - w.k_begin + kDecodeStageKeys - 1) / kDecodeStageKeys);
        return w;
    };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int st = 0; st < L::kStages; ++st) { mbar_init(full_bar(st), 1); mbar_init(empty_bar(st), 2); }
        fence_mbar_init();
    }
    __syncthreads();

    int n_issued = 0;                                                   // producer lane: stages requested so far
    if (warp == kDecodeConsumerWarps) {
        // ---- producer: one lane keeps the ring full, across the CTA's work items ----
        if (lane == 0) {
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            for (int it = blockIdx.x; it < n_items && *abort_flag == 0; it += gridDim.x) {
                const Item w = item_of(it);
                // paged cache: the page of a stage's 64 positions comes from the sequence's block table; the
                // entry of the next stage is requested before this stage's wait, so its latency is hidden
                const int* table = p.block_table ? p.block_table + size_t(w.b) * p.max_blocks : nullptr;
                int page_next = (table && w.n_stage > 0) ? table[w.k_begin / p.page_size] : 0;
                for (int i = 0; i < w.n_stage; ++i) {
                    const int gi = n_issued;
                    const int st = gi % L::kStages;
                    const int t0 = w.k_begin + i * kDecodeStageKeys;
                    const int page = page_next;
                    if (table && i + 1 < w.n_stage) page_next = table[(t0 + kDecodeStageKeys) / p.page_size];
                    if (gi >= L::kStages) mbar_wait(empty_bar(st), ((gi / L::kStages) - 1) & 1, abort_flag, 70);
                    if (*abort_flag != 0) break;
                    const uint32_t dst = smem_u32(smem + L::kRing + st * L::kStageBytes);
                    mbar_arrive_expect_tx(full_bar(st), L::kStageBytes);
                    const int c2 = table ? t0 % p.page_size : t0;          // position inside the page / the sequence
                    const int c3 = table ? page : w.b;                     // page / batch index
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        tma_load_4d(dst + h * kBoxBytes, &mapK, full_bar(st), 64 * h, w.hk / p.kv_rep, c2, c3);
                        tma_load_4d(dst + (NH + h) * kBoxBytes, &mapV, full_bar(st), 64 * h, w.hk / p.kv_rep, c2, c3);
                    }
                    n_issued = gi + 1;
                }
            }
        }
    } else {
        // ---- consumers: warp pair `pair` takes the stages whose running index is pair mod 4 (always the
        //      same ring slots); this warp its `half` (32 keys) of a stage's 64 keys ----
        // Warp-level MMA m16n8k16 with the G <= 8 heads as rows 0..7 of the 16-row operand (rows 8..15
        // are zero).  Lane = (g, t) = (lane / 4, lane % 4): g is the head for A / C rows and the key or
        // feature for B columns.
        const int pair = warp >> 1, half = warp & 1;
        const int g = lane >> 2, t = lane & 3;
        const int ctid = threadIdx.x;                                    // 0 .. 255
        // q rows (bf16, heads 0..7, zero beyond G) of an item: one 16-byte piece per thread
        auto fetch_q = [&](const Item& w) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            const int row = ctid / CH, piece = ctid % CH;
            if (ctid < 8 * CH && row < G)
                v = *reinterpret_cast<const uint4*>(p.q + (size_t(w.b) * p.H + w.hk * G + row) * D + piece * 8);
            return v;
        };
        auto store_q = [&](int buf, const uint4& v) {
            if (ctid < 8 * CH) s_qbuf[buf * 8 * CH + ctid] = v;
        };
        int qb = 0;
        int gi0 = 0;                                                     // running stage index at the start of the item
        if (blockIdx.x < n_items) store_q(0, fetch_q(item_of(blockIdx.x)));
        decode_consumer_sync();
#pragma unroll 1
        for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
            const Item w = item_of(it);
            const bool has_next = it + gridDim.x < n_items;
            uint4 qnext = make_uint4(0u, 0u, 0u, 0u);
            if (has_next) qnext = fetch_q(item_of(it + gridDim.x));       // lands while this item is processed
            // A fragments of q: for every 32 features, this lane's 8 features of head g (the same 8 features
            // that it takes from a key row below, so the pairing inside the MMA is consistent)
            uint4 qf[D / 32];
#pragma unroll
            for (int kp = 0; kp < D / 32; ++kp) qf[kp] = s_qbuf[qb * 8 * CH + g * CH + 4 * kp + t];

            float m_run = -INFINITY, lsum = 0.f;                         // of head g (same in the 4 lanes of a quad, lsum partial)
            float o[D / 8][4];                                           // [feature block][c0 c1: head g, features 2t, 2t+1; c2 c3 unused rows]
#pragma unroll
            for (int fb = 0; fb < D / 8; ++fb) { o[fb][0] = 0.f; o[fb][1] = 0.f; o[fb][2] = 0.f; o[fb][3] = 0.f; }

            const int first = (pair - (gi0 % kDecodePairs) + kDecodePairs) % kDecodePairs;
#pragma unroll 1
            for (int i = first; i < w.n_stage; i += kDecodePairs) {
                const int gi = gi0 + i;
                const int st = gi % L::kStages;
                mbar_wait(full_bar(st), (gi / L::kStages) & 1, abort_flag, 71);
                // After a wait has given up every later wait returns at once; the loops still run to their
                // ends (without touching the data) so that all warps meet at the barriers below.
                const bool live = __shfl_sync(0xffffffffu, *abort_flag, 0) == 0;
                const int k0 = w.k_begin + i * kDecodeStageKeys + half * 32;   // first key of this warp
                const int n = min(32, w.k_end - k0);                           // <= 0: second half of a short last stage
                if (live && n > 0) {
                    uint8_t* sK = smem + L::kRing + st * L::kStageBytes;
                    uint8_t* sV = sK + NH * kBoxBytes;
                    if (n < 32) {
                        // value rows past the end may hold anything (even NaN): zero them, their weights are 0
                        for (int idx = lane; idx < (32 - n) * CH; idx += 32) {
                            const int row = half * 32 + n + idx / CH, piece = idx % CH;
                            *reinterpret_cast<uint4*>(sV + (piece >> 3) * kBoxBytes + row * 128 + ((piece & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                        }
                        __syncwarp();
                    }
                    // ---- scores S[head g][key] for the 4 blocks of 8 keys ----
                    float sc[4][2];
#pragma unroll
                    for (int nb = 0; nb < 4; ++nb) {
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
                        const int r = half * 32 + 8 * nb + g;                  // B column g = key row r of the stage
#pragma unroll
                        for (int kp = 0; kp < D / 32; ++kp) {
                            const int piece = 4 * kp + t;
                            const uint4 kv = *reinterpret_cast<const uint4*>(sK + (piece >> 3) * kBoxBytes + r * 128 + (((piece & 7) ^ (r & 7)) << 4));
                            mma_bf16_16x8x16(c, qf[kp].x, 0u, qf[kp].y, 0u, kv.x, kv.y);
                            mma_bf16_16x8x16(c, qf[kp].z, 0u, qf[kp].w, 0u, kv.z, kv.w);
                        }
                        sc[nb][0] = (8 * nb + 2 * t < n) ? c[0] * p.scale_log2 : -INFINITY;       // rows past T_kv may hold anything
                        sc[nb][1] = (8 * nb + 2 * t + 1 < n) ? c[1] * p.scale_log2 : -INFINITY;
                    }
                    // ---- online softmax of head g over these 32 keys (8 per lane, 4 lanes per head) ----
                    float mx = fmaxf(fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                                     fmaxf(fmaxf(sc[2][0], sc[2][1]), fmaxf(sc[3][0], sc[3][1])));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m_run, mx);                      // finite: the block holds at least one key
                    const float alpha = fast_exp2(m_run - m_new);              // 0 on the first block
                    m_run = m_new;
                    uint32_t pa[4];                                            // P as bf16 pairs: block nb -> keys 8 nb + 2t, + 1
                    float psum = 0.f;
#pragma unroll
                    for (int nb = 0; nb < 4; ++nb) {
                        const float p0 = fast_exp2(sc[nb][0] - m_new), p1 = fast_exp2(sc[nb][1] - m_new);
                        psum += p0 + p1;
                        pa[nb] = pack_bf16x2(p0, p1);
                    }
                    lsum = lsum * alpha + psum;
                    if (alpha != 1.f) {
#pragma unroll
                        for (int fb = 0; fb < D / 8; ++fb) { o[fb][0] *= alpha; o[fb][1] *= alpha; }
                    }
                    // ---- O[head g][feature] += P V: B fragments of V through transposing matrix loads ----
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        // lane -> row address of matrix lane / 8: keys 16 ks + 8 (mat & 1) + lane % 8, piece fb + (mat >> 1)
                        const int vrow = half * 32 + 16 * ks + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                        for (int fb = 0; fb < D / 8; fb += 2) {
                            const int piece = fb + (lane >> 4);
                            const uint32_t addr = smem_u32(sV + (piece >> 3) * kBoxBytes + vrow * 128 + (((piece & 7) ^ (vrow & 7)) << 4));
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                            mma_bf16_16x8x16(o[fb], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b0, b1);
                            mma_bf16_16x8x16(o[fb + 1], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b2, b3);
                        }
                    }
                }
                // the stage is refilled by the async proxy: order this warp's accesses before the arrival
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar(st));
            }
            gi0 += w.n_stage;

            // ---- merge the eight warps, write the item's partial ----
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            if (g < G) {
                if (t == 0) { s_m[warp * G + g] = m_run; s_l[warp * G + g] = lsum; }
#pragma unroll
                for (int fb = 0; fb < D / 8; ++fb)
                    *reinterpret_cast<float2*>(&s_o[(warp * G + g) * D + 8 * fb + 2 * t]) = make_float2(o[fb][0], o[fb][1]);
            }
            if (has_next) store_q(qb ^ 1, qnext);
            decode_consumer_sync();
            float* out = p.part + ((size_t(w.b) * p.Hk + w.hk) * p.S + w.split) * G * (D + 2);
            for (int e = ctid; e < G * D; e += kDecodeConsumerThreads) {
                const int hg = e / D, c = e - hg * D;
                float mx = -INFINITY;
#pragma unroll
                for (int ww = 0; ww < kDecodeConsumerWarps; ++ww) mx = fmaxf(mx, s_m[ww * G + hg]);
                float acc = 0.f, lt = 0.f;
#pragma unroll
                for (int ww = 0; ww < kDecodeConsumerWarps; ++ww) {
                    const float f = s_m[ww * G + hg] == -INFINITY ? 0.f : fast_exp2(s_m[ww * G + hg] - mx);   // a warp without keys
                    acc = fmaf(f, s_o[(ww * G + hg) * D + c], acc);
                    lt = fmaf(f, s_l[ww * G + hg], lt);
                }
                out[hg * (D + 2) + 2 + c] = acc;
                if (c == 0) { out[hg * (D + 2)] = mx; out[hg * (D + 2) + 1] = lt; }
            }
            decode_consumer_sync();                                       // s_o, s_m, s_l free again; the next q is visible
            qb ^= 1;
        }
    }

    __syncthreads();
    if (*abort_flag != 0 && threadIdx.x == kDecodeConsumerThreads) {
        // a wait gave up: the copies requested last may still be in flight; let them land (bounded wait on
        // the latest use of each slot) before the CTA's shared memory is released
        for (int i = max(0, n_issued - L::kStages); i < n_issued; ++i)
            for (int spin = 0; spin < (1 << 20); ++spin)
                if (mbar_try_wait(full_bar(i % L::kStages), (i / L::kStages) & 1)) break;
    }
}

// One CTA of four warps per (b, query head).  Lanes hold D / 32 adjacent features; a warp takes every
// fourth depth slot and every fourth split, several of them in flight at once (the kernel is a chain
// of short dependent phases, so its time is load latency, not bandwidth).
constexpr int kDecodeMergeThreads = 128;

template <int D>
__global__ void __launch_bounds__(kDecodeMergeThreads)
decode_merge_kernel(const DecodeParams p) {
    constexpr int FPL = D / 32, NW = kDecodeMergeThreads / 32, UN = 4;
    __shared__ float s_w[kDecodeMaxSplits];          // weight of each split's partial
    __shared__ float s_d[256];                       // depth scores (log2 domain), then weights; l <= 256
    __shared__ float s_red[NW];
    __shared__ __align__(16) float s_acc[NW][D];
    const int h = blockIdx.x, b = blockIdx.y;
    const int G = p.H / p.Hk, hk = h / G, g = h - hk * G;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // this lane's features of a bf16 row, as floats
    auto load_row = [&](const __nv_bfloat16* row, float (&x)[FPL]) {
        if constexpr (FPL == 4) {
            const uint2 v = *reinterpret_cast<const uint2*>(row + lane * 4);
            x[0] = bf16_lo_to_f32(v.x); x[1] = bf16_hi_to_f32(v.x); x[2] = bf16_lo_to_f32(v.y); x[3] = bf16_hi_to_f32(v.y);
        } else {
            const uint32_t v = *reinterpret_cast<const uint32_t*>(row + lane * 2);
            x[0] = bf16_lo_to_f32(v); x[1] = bf16_hi_to_f32(v);
        }
    };
    float q[FPL];
    load_row(p.q + (size_t(b) * p.H + h) * D, q);
#pragma unroll
    for (int c = 0; c < FPL; ++c) q[c] *= p.scale_log2;
    const size_t slot_stride = size_t(p.B) * (p.Hk / p.kv_rep) * 2 * D;             // elements between depth slots
    const int Hk_real = p.Hk / p.kv_rep;                                            // p.Hk counts groups of at most 8 heads
    const __nv_bfloat16* depth0 = p.depth + (size_t(b) * Hk_real + hk / p.kv_rep) * 2 * D;   // slot 0: key row, value row at + D

    // ---- depth scores: warp `warp` takes slots warp, warp + 4, ..., UN at a time ----
    for (int i0 = warp; i0 < p.l; i0 += NW * UN) {
        float kd[UN][FPL];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int i = min(i0 + u * NW, p.l - 1);
            load_row(depth0 + size_t(i) * slot_stride, kd[u]);
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            float a = 0.f;
#pragma unroll
            for (int c = 0; c < FPL; ++c) a = fmaf(q[c], kd[u][c], a);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            if (lane == 0 && i0 + u * NW < p.l) s_d[i0 + u * NW] = a;
        }
    }
    __syncthreads();
    const float* part = p.part + ((size_t(b) * p.Hk + hk) * p.S * G + g) * (D + 2);   // + split * G * (D + 2)
    const size_t split_stride = size_t(G) * (D + 2);
    // ---- global maximum over the split maxima and the depth scores ----
    float mx = -INFINITY;
    for (int s = tid; s < p.S; s += kDecodeMergeThreads) mx = fmaxf(mx, part[s * split_stride]);
    for (int i = tid; i < p.l; i += kDecodeMergeThreads) mx = fmaxf(mx, s_d[i]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = s_red[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) mx = fmaxf(mx, s_red[w]);
    __syncthreads();
    // ---- weights and the row sum ----
    float lt = 0.f;
    for (int s = tid; s < p.S; s += kDecodeMergeThreads) {
        const float ms = part[s * split_stride];
        const float f = ms == -INFINITY ? 0.f : fast_exp2(ms - mx);
        s_w[s] = f;
        lt = fmaf(f, part[s * split_stride + 1], lt);
    }
    for (int i = tid; i < p.l; i += kDecodeMergeThreads) {
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
    // ---- weighted sum of the split partials and of the depth values: a warp takes every fourth of each ----
    float acc[FPL];
#pragma unroll
    for (int c = 0; c < FPL; ++c) acc[c] = 0.f;
    for (int s0 = warp; s0 < p.S; s0 += NW * UN) {
        float x[UN][FPL];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int s = min(s0 + u * NW, p.S - 1);
            const float* src = part + s * split_stride + 2 + lane * FPL;
#pragma unroll
            for (int c = 0; c < FPL; ++c) x[u][c] = src[c];
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const float w = s0 + u * NW < p.S ? s_w[s0 + u * NW] : 0.f;
#pragma unroll
            for (int c = 0; c < FPL; ++c) acc[c] = fmaf(w, x[u][c], acc[c]);
        }
    }
    for (int i0 = warp; i0 < p.l; i0 += NW * UN) {
        float vd[UN][FPL];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int i = min(i0 + u * NW, p.l - 1);
            load_row(depth0 + size_t(i) * slot_stride + D, vd[u]);
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const float w = i0 + u * NW < p.l ? s_d[i0 + u * NW] : 0.f;
#pragma unroll
            for (int c = 0; c < FPL; ++c) acc[c] = fmaf(w, vd[u][c], acc[c]);
        }
    }
#pragma unroll
    for (int c = 0; c < FPL; ++c) s_acc[warp][lane * FPL + c] = acc[c];
    __syncthreads();
    if (tid < D) {
        float a = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) a += s_acc[w][tid];
        p.O[(size_t(b) * p.H + h) * D + tid] = __float2bfloat16(a / lt);
    }
    if (tid == 0) p.LSE[size_t(b) * p.H + h] = (mx + log2f(lt)) * kDecodeLn2;
}

}  // namespace moda
