// Depth-KV cache layout and its pack / unpack kernels ("write" step of Sec. 2.2).
//
//   cache[slot][b][h][tile][kv][chunk][row][8]   (bf16; tile = 128 positions, chunk = 8 features)
//
// A block of one (slot, b, h, tile, kv) is 128 * d bf16 = one contiguous run.  Lane = row
// reads are 512 contiguous bytes per warp, and the same block is one bulk copy.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace moda {

constexpr int kTileRows = 128;

__host__ __device__ inline int num_tiles(int T) { return (T + kTileRows - 1) / kTileRows; }

// Elements (bf16) of one (b, h, tile, kv) block, and of one whole slot.
__host__ __device__ inline size_t cache_block_elems(int d) { return size_t(kTileRows) * d; }
__host__ __device__ inline size_t cache_slot_elems(int B, int T, int H, int d) {
    return size_t(B) * H * num_tiles(T) * 2 * cache_block_elems(d);
}
// Element offset of block (slot, b, h, tile, kv).
__host__ __device__ inline size_t cache_block_offset(int B, int T, int H, int d, int slot, int b, int h, int tile, int kv) {
    return size_t(slot) * cache_slot_elems(B, T, H, d) +
           (((size_t(b) * H + h) * num_tiles(T) + tile) * 2 + kv) * cache_block_elems(d);
}

// One CTA moves one (b, h, tile, kv) block between [B][T][H][d] and the cache, through a
// shared-memory tile so that both the global reads and the global writes are 16-byte
// accesses on consecutive addresses across a warp.
//   kToCache = true : X -> cache (append);  false : cache -> X (unpack)
template <int D, bool kToCache>
__global__ void __launch_bounds__(256)
depth_cache_copy_kernel(uint4* __restrict__ cache_slot,            // base of the slot
                        uint4* __restrict__ Xk, uint4* __restrict__ Xv,  // [B][T][H][d]
                        int T, int H) {
    constexpr int CH = D / 8;                       // 16-byte chunks per row
    __shared__ uint4 tile[kTileRows * (CH + 1)];    // +1 chunk of padding per row
    const int ntile = num_tiles(T);
    int bid = blockIdx.x;
    const int kv = bid & 1; bid >>= 1;
    const int tl = bid % ntile; bid /= ntile;
    const int h = bid % H;
    const int b = bid / H;
    uint4* X = kv ? Xv : Xk;
    if (X == nullptr) return;
    uint4* blk = cache_slot + (((size_t(b) * H + h) * ntile + tl) * 2 + kv) * (kTileRows * CH);
    const int t0 = tl * kTileRows;
    if (kToCache) {
        for (int i = threadIdx.x; i < kTileRows * CH; i += 256) {
            const int row = i / CH, ch = i % CH;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (t0 + row < T) v = X[((size_t(b) * T + t0 + row) * H + h) * CH + ch];
            tile[row * (CH + 1) + ch] = v;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < kTileRows * CH; i += 256) {
            const int ch = i / kTileRows, row = i % kTileRows;
            blk[i] = tile[row * (CH + 1) + ch];
        }
    } else {
        for (int i = threadIdx.x; i < kTileRows * CH; i += 256) {
            const int ch = i / kTileRows, row = i % kTileRows;
            tile[row * (CH + 1) + ch] = blk[i];
        }
        __syncthreads();
        for (int i = threadIdx.x; i < kTileRows * CH; i += 256) {
            const int row = i / CH, ch = i % CH;
            if (t0 + row < T) X[((size_t(b) * T + t0 + row) * H + h) * CH + ch] = tile[row * (CH + 1) + ch];
        }
    }
}

// ---- position-major layout (for grouped-query calls whose depth part runs per position) ----
//
//   cache_pm[slot][b][h][t][kv][d]   (bf16; t runs over whole 128-position tiles, tail rows zero)
//
// The K row and the V row of one position are 4 d contiguous bytes, and consecutive positions follow: the
// per-position kernels (moda_depth_gqa.cuh), which consume all rows of a few positions, read and write runs of
// (positions per CTA) * 4 d bytes per slot instead of 16-byte pieces at 2 KiB strides.  A slot has the same
// size as in the row-interleaved layout.
__host__ __device__ inline size_t cache_pm_offset(int B, int T, int H, int d, int slot, int b, int h, int t) {
    return size_t(slot) * cache_slot_elems(B, T, H, d) +
           ((size_t(b) * H + h) * (size_t(num_tiles(T)) * kTileRows) + t) * 2 * d;
}

// Grid-stride copy between [B][T][H][d] tensors and one slot of the position-major cache, 16 bytes per thread:
// consecutive threads take consecutive pieces of the cache side (K row, V row of a position).
template <int D, bool kToCache>
__global__ void __launch_bounds__(256)
depth_cache_pm_copy_kernel(uint4* __restrict__ slot_base, uint4* __restrict__ Xk, uint4* __restrict__ Xv, int B, int T, int H) {
    constexpr int CH = D / 8;
    const size_t Tp = size_t(num_tiles(T)) * kTileRows;
    const size_t total = size_t(B) * H * Tp * 2 * CH;
    for (size_t i = size_t(blockIdx.x) * 256 + threadIdx.x; i < total; i += size_t(gridDim.x) * 256) {
        const int ch = int(i % CH);
        const int kv = int((i / CH) & 1);
        const size_t row = i / (2 * CH);                 // (b * H + h) * Tp + t
        const size_t t = row % Tp, bh = row / Tp;
        const int h = int(bh % H);
        const size_t b = bh / H;
        uint4* X = kv ? Xv : Xk;
        if (kToCache) {
            uint4 v = make_uint4(0, 0, 0, 0);
            if (t < size_t(T)) v = X[((b * T + t) * H + h) * CH + ch];
            slot_base[i] = v;
        } else if (X != nullptr && t < size_t(T)) {
            X[((b * T + t) * H + h) * CH + ch] = slot_base[i];
        }
    }
}

}  // namespace moda

// =====================================================================================
// Lower-precision depth cache: e4m3 codes with one fp32 scale per row
// =====================================================================================
// (The paper's Discussion names cheaper depth-KV caching as a direction and gives no algorithm; the format
// here -- scale = max|x| / 448 per (slot, position, head, K or V) row, codes = round-to-nearest-even of
// x / scale, both in fp32 -- is this library's reading.)
//
//   cache8[slot][b][h][tile][kv] = { codes[chunk = d/16][row 128][16 bytes], scales[row 128] fp32 }
//
// A block is one contiguous run of 128 d + 512 bytes: 128 d bytes of codes in the same chunk-major, row-interleaved
// order as the bf16 cache (a chunk now holds 16 features), then the 128 row scales.
namespace moda {

__host__ __device__ inline size_t cache8_block_bytes(int d) { return size_t(kTileRows) * d + size_t(kTileRows) * 4; }
__host__ __device__ inline size_t cache8_slot_bytes(int B, int T, int H, int d) {
    return size_t(B) * H * num_tiles(T) * 2 * cache8_block_bytes(d);
}

// Correctly rounded x / scale for many x and one scale (the quantisers divide every element of a row by the row's scale,
// and the codes must be those of the IEEE quotient).  With r = RN(1 / scale):  q0 = RN(x r),  e = x - q0 scale (exact in
// one fused multiply-add),  q = RN(q0 + e r)  is the correctly rounded quotient (Markstein's division theorem) as long
// as r is within half an ulp of 1 / scale, which fails only for a significand of all ones, and nothing underflows on the
// way; both cases take the IEEE division instead (scales below 2^-80 are rows of values below 2^-71).  Quotients of
// magnitude below 2^-10 become code 0 whatever their last bit is.  Three instructions per element instead of a division.
struct RowDivider {
    float scale, r;
    bool slow;
};
__device__ __forceinline__ RowDivider make_row_divider(float scale) {
    RowDivider d;
    d.scale = scale;
    d.slow = !(scale >= 8.271806125530277e-25f) || (__float_as_uint(scale) & 0x7fffffu) == 0x7fffffu;
    d.r = d.slow ? 0.f : __frcp_rn(scale);
    return d;
}
__device__ __forceinline__ float div_rn(float x, const RowDivider& d) {
    if (d.slow) return __fdiv_rn(x, d.scale);
    const float q0 = x * d.r;
    const float e = fmaf(-q0, d.scale, x);
    return q0 == 0.f ? q0 : fmaf(e, d.r, q0);      // a zero keeps the sign of x, as the IEEE quotient does (-0 has its own code)
}

// One CTA quantises one (b, h, tile, kv) block of a [B][T][H][d] tensor into a slot.  256 threads: thread
// (row r, half hf) owns d/2 features of its row; the two halves of a row meet in shared memory for the row maximum.
template <int D>
__global__ void __launch_bounds__(256)
depth_cache_quant_kernel(uint8_t* __restrict__ slot_base, const uint4* __restrict__ Xk, const uint4* __restrict__ Xv, int T, int H) {
    constexpr int CH = D / 8;                       // 16-byte chunks (8 bf16) per input row
    __shared__ uint4 tile[kTileRows * (CH + 1)];
    __shared__ float amax2[2][kTileRows];
    const int ntile = num_tiles(T);
    int bid = blockIdx.x;
    const int kv = bid & 1; bid >>= 1;
    const int tl = bid % ntile; bid /= ntile;
    const int h = bid % H;
    const int b = bid / H;
    const uint4* X = kv ? Xv : Xk;
    uint8_t* blk = slot_base + (((size_t(b) * H + h) * ntile + tl) * 2 + kv) * cache8_block_bytes(D);
    const int t0 = tl * kTileRows;
    for (int i = threadIdx.x; i < kTileRows * CH; i += 256) {
        const int row = i / CH, ch = i % CH;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (t0 + row < T) v = X[((size_t(b) * T + t0 + row) * H + h) * CH + ch];
        tile[row * (CH + 1) + ch] = v;
    }
    __syncthreads();
    const int r = threadIdx.x & 127, hf = threadIdx.x >> 7;
    constexpr int HCH = CH / 2;                     // input chunks of this thread's half row
    float x[D / 2];
#pragma unroll
    for (int c = 0; c < HCH; ++c) {
        const uint4 v = tile[r * (CH + 1) + hf * HCH + c];
        x[8 * c + 0] = __uint_as_float(v.x << 16); x[8 * c + 1] = __uint_as_float(v.x & 0xffff0000u);
        x[8 * c + 2] = __uint_as_float(v.y << 16); x[8 * c + 3] = __uint_as_float(v.y & 0xffff0000u);
        x[8 * c + 4] = __uint_as_float(v.z << 16); x[8 * c + 5] = __uint_as_float(v.z & 0xffff0000u);
        x[8 * c + 6] = __uint_as_float(v.w << 16); x[8 * c + 7] = __uint_as_float(v.w & 0xffff0000u);
    }
    float am = 0.f;
#pragma unroll
    for (int i = 0; i < D / 2; ++i) am = fmaxf(am, fabsf(x[i]));
    amax2[hf][r] = am;
    __syncthreads();
    am = fmaxf(amax2[0][r], amax2[1][r]);
    const float scale = am > 0.f ? __fdiv_rn(am, 448.f) : 1.f;
    const RowDivider dv = make_row_divider(scale);
    uint4* codes = reinterpret_cast<uint4*>(blk);
#pragma unroll
    for (int g = 0; g < D / 32; ++g) {              // 16 features per output chunk
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float* xx = x + 16 * g + 4 * k;
            uint16_t lo, hi;
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(div_rn(xx[1], dv)), "f"(div_rn(xx[0], dv)));
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(div_rn(xx[3], dv)), "f"(div_rn(xx[2], dv)));
            w[k] = uint32_t(lo) | (uint32_t(hi) << 16);
        }
        codes[size_t(hf * (D / 32) + g) * kTileRows + r] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (hf == 0) reinterpret_cast<float*>(blk + size_t(kTileRows) * D)[r] = scale;
}

}  // namespace moda
