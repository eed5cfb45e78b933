// Attention mass on the depth slots (Sec. 2.2: the probabilities of the one softmax over sequence and depth keys; the
// paper's attention analysis reports how much probability heads give to depth slots, and its bounded slot buffer keeps
// the entries of highest utility):
//
//     mass[b, h, i] = sum_t  exp( scale <q_t, kd_i[t]> - LSE_t )          (LSE: the forward's output)
//
// HBM-bound: the depth keys of every slot are read once per query head (the heads of a group re-read them from L2), Q and
// LSE once.  Two launches: per (b, h, query tile) the 128 rows' probabilities are summed per slot in a fixed order, then
// one thread per (b, h, slot) adds the tiles' partial sums in tile order, so the result is reproducible bit for bit.
#pragma once

#include "moda_bwd.cuh"          // dot8_bf16
#include "moda_cache.cuh"
#include "sm100_ptx.cuh"

namespace moda {

struct MassParams {
    const __nv_bfloat16* Q;          // [B][T][H][d]
    const __nv_bfloat16* depth_kv;   // row-interleaved cache of H / G heads, >= l slots
    const float* LSE;                // [B][H][T]
    float* partial;                  // [B][H][tiles][l]
    float* mass;                     // [B][H][l]
    int B, T, H, G, l;
    float scale_log2;
};

// One CTA per (b, h, tile); d / 32 threads per row (32 features = four 16-byte chunks each), as in the backward's
// row-local kernel: a warp's loads of one chunk index cover whole 128-byte lines of the chunk-major cache block.
template <int D>
__global__ void __launch_bounds__(kTileRows * (D / 32))
depth_slot_mass_kernel(const MassParams p) {
    constexpr int PARTS = D / 32;
    constexpr int CH = D / 8;
    constexpr int kWarps = kTileRows * PARTS / 32;
    __shared__ float warp_sum[256 * kWarps];     // [slot][warp]: l <= 256 slots
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = lane % PARTS;
    const int r = warp * (32 / PARTS) + lane / PARTS;
    const int nq = num_tiles(p.T);
    const int qt = blockIdx.x % nq;
    const int bh = blockIdx.x / nq;
    const int b = bh / p.H, h = bh % p.H;
    const int Hk = p.H / p.G, hk = h / p.G;
    const int t = qt * kTileRows + r;
    const bool valid = t < p.T;

    uint4 q4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) q4[j] = make_uint4(0, 0, 0, 0);
    if (valid) {
        const uint4* Q = reinterpret_cast<const uint4*>(p.Q) + ((size_t(b) * p.T + t) * p.H + h) * CH + part * 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) q4[j] = Q[j];
    }
    const float neg_lse2 = valid ? -p.LSE[(size_t(b) * p.H + h) * p.T + t] * kLog2e : -INFINITY;   // rows past T add 0
    const size_t slot_stride = cache_slot_elems(p.B, p.T, Hk, D) / 8;                              // in uint4
    const uint4* cK = reinterpret_cast<const uint4*>(p.depth_kv) +
                      ((size_t(b) * Hk + hk) * nq + qt) * 2 * (kTileRows * CH) + size_t(part * 4) * kTileRows + r;
    float* out = p.partial + (size_t(bh) * nq + qt) * p.l;
#pragma unroll 1
    for (int i = 0; i < p.l; ++i) {
        float u = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) u += dot8_bf16(q4[j], __ldcs(cK + j * kTileRows));
#pragma unroll
        for (int off = 1; off < PARTS; off <<= 1) u += __shfl_xor_sync(0xffffffffu, u, off);
        float R = part == 0 ? fast_exp2(fmaf(u, p.scale_log2, neg_lse2)) : 0.f;
        // rows of the warp in a fixed order; the warps are added after the loop
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) R += __shfl_xor_sync(0xffffffffu, R, off);
        if (lane == 0) warp_sum[i * kWarps + warp] = R;
        cK += slot_stride;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < p.l; i += blockDim.x) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += warp_sum[i * kWarps + w];
        out[i] = s;
    }
}

// mass[b][h][i] = sum over the tiles, in tile order.
__global__ void __launch_bounds__(256)
depth_slot_mass_reduce_kernel(const MassParams p) {
    const int nq = num_tiles(p.T);
    const long long n = (long long)p.B * p.H * p.l;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    const int i = int(idx % p.l);
    const long long bh = idx / p.l;
    const float* src = p.partial + size_t(bh) * nq * p.l + i;
    float s = 0.f;
    for (int q = 0; q < nq; ++q) s += src[size_t(q) * p.l];
    p.mass[idx] = s;
}

}  // namespace moda
