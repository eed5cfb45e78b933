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

}  // namespace moda
