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

// hist: complete histogram of keys.  hist_next: a second histogram buffer that
// is cleared here for the following call (nobody reads it during this kernel).
// Dynamic shared memory: kBucketWarps * bins_per_cta ints.
__global__ void __launch_bounds__(kBucketThreads)
k_bucket(const int32_t* __restrict__ keys, const int* __restrict__ hist, int* __restrict__ hist_next,
         int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int B, int nbins, int bins_per_cta)
{
    extern __shared__ int s_cnt[];                 // [kBucketWarps][bins_per_cta]
    __shared__ int s_warp[kBucketWarps];
    __shared__ int s_base;

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int lo = blockIdx.x * bins_per_cta;
    if (lo >= nbins) return;
    const int hi = min(lo + bins_per_cta, nbins);
    const int nb = bins_per_cta;

    for (int i = tid; i < kBucketWarps * nb; i += kBucketThreads) s_cnt[i] = 0;

    // tokens in bins below this CTA's range
    int part = 0;
    for (int i = tid; i < lo; i += kBucketThreads) part += hist[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);
    if (lane == 0) s_warp[w] = part;
    __syncthreads();
    if (w == 0) {
        int v = s_warp[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
        if (lane == 0) s_base = v;
    }
    __syncthreads();

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

    // scan: first output position of every bin, then of every (warp, bin)
    {
        const int b = lo + tid;
        const int c = (tid < nb && b < hi) ? hist[b] : 0;
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(kFullMask, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_warp[w] = incl;
        __syncthreads();
        if (w == 0) {
            int v = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(kFullMask, v, o);
                if (lane >= o) v += u;
            }
            s_warp[lane] = v;                       // inclusive over warps
        }
        __syncthreads();
        const int start = s_base + (w > 0 ? s_warp[w - 1] : 0) + incl - c;
        if (tid < nb && b < hi) {
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

}  // namespace fff
