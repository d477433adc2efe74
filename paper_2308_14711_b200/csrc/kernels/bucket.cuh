// Leaf bucketing: stable counting sort of token ids by bin (leaf or node position).
//
//   offsets[j]          = number of tokens whose bin is < j      (offsets[nbins] = B)
//   perm[offsets[j]+r]  = r-th smallest token id with bin j
//
// The result is unique, so it is reproduced bit for bit.  No float, no
// order-dependent atomics: the only atomics are the integer histogram counts,
// whose sums do not depend on arrival order.
//
// Decomposition: the bins are split into contiguous ranges, one CTA per range.
// Every CTA reads all B keys (B * 4 bytes, L2-resident) and places the tokens
// of its own bins.  Inside the CTA each of the 32 warps owns a contiguous slice
// of the token ids, so "earlier token" means "earlier warp, or earlier step of
// the same warp, or lower lane of the same step" -- three orders that are all
// resolved without communication between CTAs:
//   pass 1  per-warp, per-bin counts in shared memory;
//   scan    bin starts from the global histogram, warp starts from the counts;
//   pass 2  each warp re-reads its slice in order and writes perm.
#pragma once

#include "common.cuh"

namespace fff {

constexpr int kBucketWarps = 32;
constexpr int kBucketThreads = kBucketWarps * 32;
constexpr int kBucketMaxBinsPerCta = 1024;   // one bin per thread in the scan phase

// Histogram of keys (warp-aggregated so that a hot bin costs one atomic per warp step).
__global__ void __launch_bounds__(256)
k_histogram(const int32_t* __restrict__ keys, int* __restrict__ hist, int64_t B, int nbins)
{
    const int lane = threadIdx.x & 31;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t rounds = (B + stride - 1) / stride;
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t r = 0; r < rounds; ++r, t += stride) {
        int k = t < B ? keys[t] : -1;
        const bool ok = k >= 0 && k < nbins;            // out-of-range ids are ignored
        if (!ok) k = -1 - lane;                         // idle lanes get unique dummies
        const unsigned peers = __match_any_sync(kFullMask, k);
        if (ok && lane == __ffs(peers) - 1) atomicAdd(hist + k, __popc(peers));
    }
}

// Sum over the block; every thread returns the total.  s_warp: kBucketWarps ints of scratch.
__device__ __forceinline__ int block_sum(int v, int* s_warp)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    __syncthreads();
    if (lane == 0) s_warp[w] = v;
    __syncthreads();
    int t = s_warp[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(kFullMask, t, o);
    return t;
}

// Exclusive prefix sum over the block in thread order.  s_warp: kBucketWarps ints of scratch.
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(kFullMask, incl, o);
        if (lane >= o) incl += u;
    }
    __syncthreads();
    if (lane == 31) s_warp[w] = incl;
    __syncthreads();
    int ws = s_warp[lane];                     // lane i holds the total of warp i
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(kFullMask, ws, o);
        if (lane >= o) ws += u;
    }
    const int before = __shfl_sync(kFullMask, ws, max(w - 1, 0));
    return (w > 0 ? before : 0) + incl - v;
}

// hist: complete histogram of keys.  hist_next: a second histogram buffer that
// is cleared here for the following call (nobody reads it during this kernel).
// tile_rows > 0 additionally writes the tile list of the grouped kernels: the
// tiles of bin 0 first, each bin cut into ceil(count / tile_rows) tiles, and
// their number into *n_tiles.
// Dynamic shared memory: kBucketWarps * bins_per_cta ints.
__global__ void __launch_bounds__(kBucketThreads)
k_bucket(const int32_t* __restrict__ keys, const int* __restrict__ hist, int* __restrict__ hist_next,
         int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int B, int nbins, int bins_per_cta,
         int tile_rows, Tile* __restrict__ tiles, int* __restrict__ n_tiles)
{
    extern __shared__ int s_cnt[];                 // [kBucketWarps][bins_per_cta]
    __shared__ int s_warp[kBucketWarps];

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int lo = blockIdx.x * bins_per_cta;
    if (lo >= nbins) return;
    const int hi = min(lo + bins_per_cta, nbins);
    const int nb = bins_per_cta;

    for (int i = tid; i < kBucketWarps * nb; i += kBucketThreads) s_cnt[i] = 0;

    // tokens (and tiles) in bins below this CTA's range
    int part = 0, tpart = 0;
    for (int i = tid; i < lo; i += kBucketThreads) {
        const int c = hist[i];
        part += c;
        if (tile_rows > 0) tpart += (c + tile_rows - 1) / tile_rows;
    }
    const int base = block_sum(part, s_warp);
    const int tile_base = tile_rows > 0 ? block_sum(tpart, s_warp) : 0;

    // token slice of this warp (a multiple of 32 so that steps never straddle slices)
    const int chunk = (((B + kBucketWarps - 1) / kBucketWarps) + 31) & ~31;
    const int t0 = min(w * chunk, B), t1 = min(t0 + chunk, B);
    int* my = s_cnt + w * nb;

    // pass 1: count
    for (int s = t0; s < t1; s += 32) {
        const int t = s + lane;
        const int k = t < t1 ? keys[t] : -1;
        const bool in = k >= lo && k < hi;
        const unsigned peers = __match_any_sync(kFullMask, in ? k : -1 - lane);
        if (in && lane == __ffs(peers) - 1) my[k - lo] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();

    // scan: first output position of every bin, then of every (warp, bin); tile list
    {
        const int b = lo + tid;
        const bool mine = tid < nb && b < hi;
        const int c = mine ? hist[b] : 0;
        const int start = base + block_exclusive_scan(c, s_warp);
        if (mine) {
            offsets[b] = start;
            if (b == nbins - 1) offsets[nbins] = start + c;
            int run = start;
            for (int ww = 0; ww < kBucketWarps; ++ww) {
                const int c2 = s_cnt[ww * nb + tid];
                s_cnt[ww * nb + tid] = run;
                run += c2;
            }
            hist_next[b] = 0;
        }
        if (tile_rows > 0) {
            const int nt = (c + tile_rows - 1) / tile_rows;
            const int t0 = tile_base + block_exclusive_scan(nt, s_warp);
            if (mine) {
                for (int i = 0; i < nt; ++i) {
                    Tile tl;
                    tl.bin = b;
                    tl.start = start + i * tile_rows;
                    tl.rows = min(tile_rows, c - i * tile_rows);
                    tl.pad = 0;
                    tiles[t0 + i] = tl;
                }
                if (b == nbins - 1) *n_tiles = t0 + nt;
            }
        }
    }
    __syncthreads();

    // pass 2: place
    for (int s = t0; s < t1; s += 32) {
        const int t = s + lane;
        const int k = t < t1 ? keys[t] : -1;
        const bool in = k >= lo && k < hi;
        const unsigned peers = __match_any_sync(kFullMask, in ? k : -1 - lane);
        const int leader = __ffs(peers) - 1;
        int pos = 0;
        if (in && lane == leader) {
            pos = my[k - lo];
            my[k - lo] = pos + __popc(peers);
        }
        pos = __shfl_sync(kFullMask, pos, leader);
        if (in) perm[pos + __popc(peers & ((1u << lane) - 1u))] = t;
        __syncwarp();
    }
}

// Tile list from an existing offsets array (one CTA; used when the caller supplies the bucketing).
__global__ void __launch_bounds__(kBucketThreads)
k_tiles_from_offsets(const int32_t* __restrict__ offsets, int nbins, int tile_rows, Tile* __restrict__ tiles,
                     int* __restrict__ n_tiles)
{
    __shared__ int s_warp[kBucketWarps];
    int tile_base = 0;
    for (int b0 = 0; b0 < nbins; b0 += kBucketThreads) {
        const int b = b0 + threadIdx.x;
        const int start = b < nbins ? offsets[b] : 0;
        const int c = b < nbins ? offsets[b + 1] - start : 0;
        const int nt = (c + tile_rows - 1) / tile_rows;
        const int t0 = tile_base + block_exclusive_scan(nt, s_warp);
        for (int i = 0; i < nt; ++i) {
            Tile tl;
            tl.bin = b;
            tl.start = start + i * tile_rows;
            tl.rows = min(tile_rows, c - i * tile_rows);
            tl.pad = 0;
            tiles[t0 + i] = tl;
        }
        tile_base += block_sum(nt, s_warp);
    }
    if (threadIdx.x == 0) *n_tiles = tile_base;
}

}  // namespace fff
