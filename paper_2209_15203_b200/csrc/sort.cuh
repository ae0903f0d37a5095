// Segmented stable LSD radix sort of (index, value) entries by index, 8 bits per
// pass.  It puts a message into its canonical order (ascending index); the
// selection kernels emit entries in arbitrary order because nothing on the
// per-step path depends on it.
//
// One pass = three kernels:
//   sort_local    each CTA sorts its tile of 1024 entries by the current digit
//                 (eight stable 1-bit splits in shared memory), writes the tile
//                 back and records how many entries of each digit it holds
//   sort_scan     per row: exclusive prefix over (digit-major, tile-minor) counts
//   sort_scatter  each entry goes to  prefix[digit][tile] + rank inside the tile
#pragma once

#include "common.cuh"

namespace tk {

constexpr int kSortTile = 1024;

// Stable split of the tile by one bit: zeros first.  `e` is this thread's entry,
// `valid` whether it is a real entry (invalid ones are at the end and stay there).
__device__ __forceinline__ void split_by_bit(uint2& e, bool& valid, int bit, uint2* sh_e,
                                             unsigned char* sh_valid, u32* scratch) {
    bool zero = valid && (((e.x >> bit) & 1u) == 0);
    u32 total;
    u32 incl = block_inclusive_scan(zero ? 1u : 0u, scratch, &total);
    u32 pos = zero ? incl - 1 : total + (threadIdx.x - incl);
    sh_e[pos] = e;
    sh_valid[pos] = valid ? 1 : 0;
    __syncthreads();
    e = sh_e[threadIdx.x];
    valid = sh_valid[threadIdx.x] != 0;
    __syncthreads();
}

// After the local sort, position p of the tile holds digit sh_dig[p]; returns
// the first position of this thread's digit run.
__device__ __forceinline__ u32 run_start(u32 dig, bool valid, u32* sh_dig, u32* sh_start) {
    sh_dig[threadIdx.x] = valid ? dig : 0xffffffffu;
    __syncthreads();
    if (valid && (threadIdx.x == 0 || sh_dig[threadIdx.x - 1] != dig)) sh_start[dig] = threadIdx.x;
    __syncthreads();
    return valid ? sh_start[dig] : 0;
}

__global__ void __launch_bounds__(kSortTile)
sort_local_kernel(uint2* src, size_t stride, const u32* counts, size_t count_stride, u32 n_fixed,
                  int shift, u32 tiles, u32* cnt) {
    __shared__ uint2 sh_e[kSortTile];
    __shared__ unsigned char sh_valid[kSortTile];
    __shared__ u32 sh_dig[kSortTile];
    __shared__ u32 sh_start[256];
    __shared__ u32 sh_cnt[256];
    __shared__ u32 scratch[33];
    const int row = blockIdx.y;
    const u32 tile = blockIdx.x;
    const u32 n = counts ? min(n_fixed, counts[(size_t)row * count_stride]) : n_fixed;
    uint2* seg = src + (size_t)row * stride;
    u32 i = tile * kSortTile + threadIdx.x;
    bool valid = i < n;
    uint2 e = valid ? seg[i] : make_uint2(0xffffffffu, 0);
    for (int b = 0; b < 8; ++b) split_by_bit(e, valid, shift + b, sh_e, sh_valid, scratch);
    u32 dig = (e.x >> shift) & 255u;
    if (threadIdx.x < 256) sh_cnt[threadIdx.x] = 0;
    u32 start = run_start(dig, valid, sh_dig, sh_start);
    bool last = valid && (threadIdx.x == kSortTile - 1 || sh_dig[threadIdx.x + 1] != dig);
    if (last) sh_cnt[dig] = threadIdx.x - start + 1;
    __syncthreads();
    if (threadIdx.x < 256) cnt[((size_t)row * 256 + threadIdx.x) * tiles + tile] = sh_cnt[threadIdx.x];
    if (valid) seg[i] = e;
}

__global__ void __launch_bounds__(256) sort_scan_kernel(u32* cnt, u32 tiles) {
    __shared__ u32 scratch[33];
    const int row = blockIdx.x;
    u32* c = cnt + ((size_t)row * 256 + threadIdx.x) * tiles;
    u32 sum = 0;
    for (u32 t = 0; t < tiles; ++t) sum += c[t];
    u32 total;
    u32 base = block_inclusive_scan(sum, scratch, &total) - sum;
    for (u32 t = 0; t < tiles; ++t) {
        u32 v = c[t];
        c[t] = base;
        base += v;
    }
}

// dst != NULL: write entries to dst (same stride); else split into idx_out / val_out rows of
// out_stride elements.
__global__ void __launch_bounds__(kSortTile)
sort_scatter_kernel(const uint2* src, size_t stride, const u32* counts, size_t count_stride,
                    u32 n_fixed, int shift, u32 tiles, const u32* cnt, uint2* dst,
                    int32_t* idx_out, float* val_out, size_t out_stride) {
    __shared__ u32 sh_dig[kSortTile];
    __shared__ u32 sh_start[256];
    const int row = blockIdx.y;
    const u32 tile = blockIdx.x;
    const u32 n = counts ? min(n_fixed, counts[(size_t)row * count_stride]) : n_fixed;
    const uint2* seg = src + (size_t)row * stride;
    u32 i = tile * kSortTile + threadIdx.x;
    bool valid = i < n;
    uint2 e = valid ? seg[i] : make_uint2(0xffffffffu, 0);
    u32 dig = (e.x >> shift) & 255u;
    u32 start = run_start(dig, valid, sh_dig, sh_start);
    if (!valid) return;
    u32 pos = cnt[((size_t)row * 256 + dig) * tiles + tile] + (threadIdx.x - start);
    if (dst) {
        dst[(size_t)row * stride + pos] = e;
    } else {
        idx_out[(size_t)row * out_stride + pos] = (int32_t)e.x;
        val_out[(size_t)row * out_stride + pos] = __uint_as_float(e.y);
    }
}

}  // namespace tk
