// Exclusive prefix sums over device arrays (three small kernels: tile sums,
// scan of the tile sums, rescan with offsets).  out has n + 1 entries.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mlip {

constexpr int SCAN_THREADS = 1024;
constexpr int SCAN_ITEMS = 4;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

// Exclusive scan of one value per thread across a 1024-thread block.
__device__ __forceinline__ int64_t block_exclusive_scan(int64_t v, int64_t &total, int64_t *warp_sums /* [32] shared */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int64_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int64_t w = warp_sums[lane], wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int64_t t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sums[lane] = wi - w;   // exclusive offsets of the warps
        if (lane == 31) warp_sums[32] = wi;
    }
    __syncthreads();
    total = warp_sums[32];
    int64_t r = warp_sums[warp] + incl - v;
    __syncthreads();
    return r;
}

template <typename TIn>
__global__ void __launch_bounds__(SCAN_THREADS) scan_tile_sums(const TIn *__restrict__ in, int64_t n, int64_t *__restrict__ sums) {
    __shared__ int64_t ws[33];
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int64_t v = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i)
        if (base + i < n) v += (int64_t)in[base + i];
    int64_t total;
    block_exclusive_scan(v, total, ws);
    if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// One block: exclusive scan of the tile sums in place; sums[nb] receives the grand total.
static __global__ void __launch_bounds__(SCAN_THREADS) scan_of_sums(int64_t *sums, int64_t nb) {
    __shared__ int64_t ws[33];
    int64_t carry = 0;
    for (int64_t base = 0; base < nb; base += SCAN_THREADS) {
        int64_t idx = base + threadIdx.x;
        int64_t v = idx < nb ? sums[idx] : 0, total;
        int64_t ex = block_exclusive_scan(v, total, ws);
        if (idx < nb) sums[idx] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) sums[nb] = carry;
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(SCAN_THREADS) scan_apply(const TIn *__restrict__ in, TOut *__restrict__ out, int64_t n,
                                                           const int64_t *__restrict__ sums, int64_t nb) {
    __shared__ int64_t ws[33];
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int64_t item[SCAN_ITEMS], v = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        item[i] = base + i < n ? (int64_t)in[base + i] : 0;
        v += item[i];
    }
    int64_t total;
    int64_t run = sums[blockIdx.x] + block_exclusive_scan(v, total, ws);
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (base + i < n) out[base + i] = (TOut)run;
        run += item[i];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) out[n] = (TOut)sums[nb];
}

// Enqueue an exclusive scan; `tmp` must hold n / SCAN_TILE + 2 int64 values.
template <typename TIn, typename TOut>
inline void exclusive_scan(const TIn *in, TOut *out, int64_t n, int64_t *tmp, cudaStream_t s) {
    int64_t nb = (n + SCAN_TILE - 1) / SCAN_TILE;
    if (nb < 1) nb = 1;
    scan_tile_sums<TIn><<<(unsigned)nb, SCAN_THREADS, 0, s>>>(in, n, tmp);
    scan_of_sums<<<1, SCAN_THREADS, 0, s>>>(tmp, nb);
    scan_apply<TIn, TOut><<<(unsigned)nb, SCAN_THREADS, 0, s>>>(in, out, n, tmp, nb);
}

inline int64_t scan_tmp_items(int64_t n) { return n / SCAN_TILE + 3; }

}  // namespace mlip
