// Leaf bucketing: stable counting sort of token ids by bin (leaf or node position).
//
//   offsets[j]          = number of tokens whose bin is < j      (offsets[nbins] = B)
//   perm[offsets[j]+r]  = r-th smallest token id with bin j
//
// The result is unique (tokens of a bin stay in token order), so every kernel here reproduces it bit for
// bit.  No float, and no atomics whose arrival order could show in the result: the integer sums that
// some variants accumulate atomically do not depend on it.
//
// Four implementations of the same sort, chosen by the caller:
//   k_histogram + k_bucket    two launches; the bins are split into contiguous ranges, one CTA per range
//                             reads all keys and places the tokens of its bins (the allocation-free
//                             entry point uses these: their only scratch is the histogram);
//   k_bucket_cluster          one launch, clusters of 8 CTAs exchange per-CTA counts through distributed
//                             shared memory; global mode (every cluster scans all keys for its bin range)
//                             or segmented mode (one cluster per bucket of a previous, coarser bucketing);
//   k_bucket_coop             one cooperative launch for up to 1024 bins: every CTA ranks one slice of the
//                             tokens, one grid-wide barrier, column sums over the per-CTA counts;
//   k_bucket_ranked           after the first descent stage, whose epilogue has already ranked the tokens of
//                             each 128-token tile: sum of the per-tile counts, scan, scatter; no barrier
//                             across CTAs.
// In all of them "earlier token" is resolved hierarchically: earlier slice (tile, CTA, warp), earlier step of
// the same warp, lower lane of the same step (ballot masks of equal keys).
// Each can also write the tile list of the grouped kernel that follows: the tiles of bin 0 first, each bin
// cut into tiles of at most tile_rows consecutive entries, padded with empty tiles to a length the host knows.
#pragma once

#include <cooperative_groups.h>

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

// hist: complete histogram of keys.  hist_next: a second histogram buffer whose
// first nbins counters are cleared here (nobody reads it during this kernel).
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

// ---- cluster version ---------------------------------------------------------------------------
// Self-contained stable bucketing: no histogram input, no atomics.
//
// A thread-block cluster of 8 CTAs owns one contiguous range of bins and one list of candidate
// tokens; it counts, scans and places on its own:
//   * global mode (seg_offsets == NULL): the candidates are all B tokens in natural order; cluster c
//     owns bins [c*nb, (c+1)*nb) and ignores tokens whose key falls outside (it still counts the
//     tokens with smaller keys, which gives the first output position of its range);
//   * segmented mode: the tokens were already bucketed by a coarser key (perm_in, seg_offsets) and
//     refining that order only moves tokens inside their old bucket.  Cluster c handles the tokens
//     perm_in[seg_offsets[c] .. seg_offsets[c+1]), whose keys all lie in [c*nb, (c+1)*nb), and writes
//     exactly that range of perm_out.  Work is spread over all old buckets at once.
// The candidate list is split into 8 * NW contiguous slices, one per warp of the cluster.  Each warp
// makes one matching pass over its slice (keys in registers when the slice has at most
// 32 * kBucketKeyRegs tokens, else the per-token rank goes through `rank_tmp`), per-CTA totals are
// exchanged through distributed shared memory, and a second trivial pass writes perm_out.
//
// Tile list (tile_rows > 0): cluster c writes the tiles of its bins starting at entry
// floor(first_position / tile_rows) + c*nb -- an upper bound of the number of tiles before it -- and
// pads its region up to the next cluster's start with empty tiles (rows = 0), so that the list has a
// size known on the host, n_tiles_total = floor(B / tile_rows) + nbins, and needs no global scan.
constexpr int kBucketClusterSize = 8;
constexpr int kBucketKeyRegs = 8;

// Lanes holding the same value v (only the low nbits bits may differ) among the lanes with `in` set;
// built from one ballot per bit, which is far cheaper than the match instruction when a whole SM
// issues it at once.  The result is only meaningful for lanes with `in` set.
__device__ __forceinline__ unsigned peers_by_ballot(bool in, int v, int nbits)
{
    unsigned peers = __ballot_sync(kFullMask, in);
    for (int bit = 0; bit < nbits; ++bit) {
        const bool one = (v >> bit) & 1;
        const unsigned m = __ballot_sync(kFullMask, one);
        peers &= one ? m : ~m;
    }
    return peers;
}

template <int NW> __device__ __forceinline__ int block_sum_nw(int v, int* s_warp)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    __syncthreads();
    if (lane == 0) s_warp[w] = v;
    __syncthreads();
    int t = lane < NW ? s_warp[lane] : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(kFullMask, t, o);
    return t;
}

// Exclusive prefix sum over the block in thread order; *total receives the block total.
template <int NW> __device__ __forceinline__ int block_exclusive_scan_nw(int v, int* s_warp, int* total)
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
    int ws = lane < NW ? s_warp[lane] : 0;        // lane i holds the total of warp i
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(kFullMask, ws, o);
        if (lane >= o) ws += u;
    }
    *total = __shfl_sync(kFullMask, ws, NW - 1);
    const int before = __shfl_sync(kFullMask, ws, max(w - 1, 0));
    return (w > 0 ? before : 0) + incl - v;
}

// Dynamic shared memory: (NW + 1) * nb ints.  Requires nb <= NW * 32.
template <int NW>
__global__ void __launch_bounds__(NW * 32, NW == 32 ? 1 : 4)
k_bucket_cluster(const int32_t* __restrict__ keys, const int32_t* __restrict__ perm_in,
                 const int32_t* __restrict__ seg_offsets, int32_t* __restrict__ offsets_out,
                 int32_t* __restrict__ perm_out, int B, int nbins, int nb, int bin_bits, int tile_rows,
                 Tile* __restrict__ tiles, int n_tiles_total, int32_t* __restrict__ rank_tmp)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int kThreads = NW * 32;
    extern __shared__ int s_dyn[];
    __shared__ int s_warp[32];
    __shared__ int s_below;                          // tokens of this CTA's slices with a key below the range

    int* s_cnt = s_dyn;                              // [NW][nb]
    int* s_tot = s_dyn + NW * nb;                    // [nb] tokens of this CTA's slices per bin (read by peers)
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int rank = (int)cluster.block_rank();
    const int c = blockIdx.x / kBucketClusterSize;
    const int n_clusters = gridDim.x / kBucketClusterSize;
    const int lo = c * nb, hi = min(lo + nb, nbins);
    pdl_trigger();
    pdl_wait();
    const int seg_lo = seg_offsets ? seg_offsets[c] : 0;
    const int seg_hi = seg_offsets ? seg_offsets[c + 1] : B;
    const unsigned lt_mask = (1u << lane) - 1u;

    for (int i = tid; i < NW * nb; i += kThreads) s_cnt[i] = 0;
    __syncthreads();

    const int slices = kBucketClusterSize * NW;
    const int chunk = ((((seg_hi - seg_lo) + slices - 1) / slices) + 31) & ~31;
    const int t0 = min(seg_lo + (rank * NW + w) * chunk, seg_hi), t1 = min(t0 + chunk, seg_hi);
    const bool in_regs = chunk <= 32 * kBucketKeyRegs;       // uniform over the cluster
    int* my = s_cnt + w * nb;

    // pass 1: count and rank inside the slice
    int kreg[kBucketKeyRegs], rreg[kBucketKeyRegs], treg[kBucketKeyRegs];
#pragma unroll
    for (int i = 0; i < kBucketKeyRegs; ++i) { kreg[i] = -1; rreg[i] = 0; treg[i] = 0; }
    int below = 0;
    for (int s0 = t0; s0 < t1; s0 += 32 * kBucketKeyRegs) {
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            const int idx = s0 + i * 32 + lane;
            treg[i] = idx < t1 ? (perm_in ? __ldg(perm_in + idx) : idx) : -1;
        }
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) kreg[i] = treg[i] >= 0 ? __ldg(keys + treg[i]) : -1;
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            if (s0 + i * 32 >= t1) break;
            const int k = kreg[i];
            const bool in = k >= lo && k < hi;
            below += (k >= 0 && k < lo) ? 1 : 0;
            const unsigned peers = peers_by_ballot(in, k - lo, bin_bits);
            const int leader = in ? __ffs(peers) - 1 : lane;
            int seen = 0;
            if (in && lane == leader) {
                seen = my[k - lo];
                my[k - lo] = seen + __popc(peers);
            }
            seen = __shfl_sync(kFullMask, seen, leader) + __popc(peers & lt_mask);
            if (in_regs) rreg[i] = seen;
            else if (in) rank_tmp[s0 + i * 32 + lane] = seen;
            __syncwarp();
        }
    }
    const int below_cta = seg_offsets ? 0 : block_sum_nw<NW>(below, s_warp);
    __syncthreads();

    // per bin: offsets of the warps inside this CTA, and this CTA's total
    const int b = lo + tid;
    const bool mine = tid < nb && b < hi;
    if (mine) {
        int run = 0;
        for (int ww = 0; ww < NW; ++ww) {
            const int c2 = s_cnt[ww * nb + tid];
            s_cnt[ww * nb + tid] = run;
            run += c2;
        }
        s_tot[tid] = run;
    }
    if (tid == 0) s_below = below_cta;
    cluster.sync();

    // totals over the cluster, tokens of lower-ranked CTAs, first position of every bin
    int total = 0, before = 0;
    if (mine) {
#pragma unroll
        for (int r = 0; r < kBucketClusterSize; ++r) {
            const int v = reinterpret_cast<const int*>(cluster.map_shared_rank(s_tot, r))[tid];
            total += v;
            if (r < rank) before += v;
        }
    }
    int first = seg_lo;                              // first output position of the cluster's range
    if (!seg_offsets) {
        first = 0;
#pragma unroll
        for (int r = 0; r < kBucketClusterSize; ++r) first += *reinterpret_cast<const int*>(cluster.map_shared_rank(&s_below, r));
    }
    int cluster_total = 0;
    const int start = first + block_exclusive_scan_nw<NW>(total, s_warp, &cluster_total);
    if (mine) {
        const int add = start + before;
        for (int ww = 0; ww < NW; ++ww) s_cnt[ww * nb + tid] += add;
        if (rank == 0) {
            offsets_out[b] = start;
            if (b == nbins - 1) offsets_out[nbins] = start + total;
        }
    }
    if (tile_rows > 0 && rank == 0) {
        const int nt = (total + tile_rows - 1) / tile_rows;
        int n_mine = 0;
        const int region = first / tile_rows + lo;
        const int tl0 = region + block_exclusive_scan_nw<NW>(nt, s_warp, &n_mine);
        if (mine) {
            for (int i = 0; i < nt; ++i) {
                Tile tl;
                tl.bin = b;
                tl.start = start + i * tile_rows;
                tl.rows = min(tile_rows, total - i * tile_rows);
                tl.pad = 0;
                tiles[tl0 + i] = tl;
            }
        }
        const int region_end = c == n_clusters - 1 ? n_tiles_total : (first + cluster_total) / tile_rows + hi;
        Tile empty;
        empty.bin = 0; empty.start = 0; empty.rows = 0; empty.pad = 0;
        for (int i = region + n_mine + tid; i < region_end; i += kThreads) tiles[i] = empty;
    }
    __syncthreads();

    // pass 2: place
    if (in_regs) {
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            const int k = kreg[i];
            if (k >= lo && k < hi) perm_out[my[k - lo] + rreg[i]] = treg[i];
        }
    } else {
        for (int idx = t0 + lane; idx < t1; idx += 32) {
            const int t = perm_in ? __ldg(perm_in + idx) : idx;
            const int k = __ldg(keys + t);
            if (k >= lo && k < hi) perm_out[my[k - lo] + rank_tmp[idx]] = t;
        }
    }
    cluster.sync();      // peers may still be reading this CTA's shared memory
}

// ---- grid-wide version for few bins ----------------------------------------------------------------
// Global bucketing (all B tokens in natural order) of at most kBucketMaxBinsPerCta bins with the work
// spread over the whole GPU: CTA c of G takes the c-th contiguous slice of the tokens, counts per
// (warp, bin), publishes its per-bin totals as row c of a G x nbins matrix in global memory, and after
// one grid-wide barrier (cooperative launch; all CTAs are resident) adds up the rows of the CTAs before
// it.  Same result as k_bucket_cluster, which needs one cluster (8 SMs) to scan every token.
// The tile list is written dense and padded with empty tiles up to n_tiles_total.
constexpr int kCoopWarps = 8;
constexpr int kCoopThreads = kCoopWarps * 32;

// Dynamic shared memory: (kCoopWarps + 2) * nbins ints.
__global__ void __launch_bounds__(kCoopThreads)
k_bucket_coop(const int32_t* __restrict__ keys, int32_t* __restrict__ offsets_out, int32_t* __restrict__ perm_out, int B,
              int nbins, int bin_bits, int tile_rows, Tile* __restrict__ tiles, int n_tiles_total,
              int32_t* __restrict__ rank_tmp, int* __restrict__ matrix)
{
    namespace cg = cooperative_groups;
    extern __shared__ int s_dyn[];
    __shared__ int s_warp[32];
    int* s_cnt = s_dyn;                              // [kCoopWarps][nbins]
    int* s_start = s_dyn + kCoopWarps * nbins;       // [nbins] first position of the bin
    int* s_total = s_start + nbins;                  // [nbins] tokens in the bin
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int G = gridDim.x, c = blockIdx.x;
    const unsigned lt_mask = (1u << lane) - 1u;

    pdl_trigger();
    for (int i = tid; i < (kCoopWarps + 2) * nbins; i += kCoopThreads) s_cnt[i] = 0;     // counts, starts and totals
    __syncthreads();
    pdl_wait();

    const int slices = G * kCoopWarps;
    const int chunk = (((B + slices - 1) / slices) + 31) & ~31;
    const int t0 = min((c * kCoopWarps + w) * chunk, B), t1 = min(t0 + chunk, B);
    const bool in_regs = chunk <= 32 * kBucketKeyRegs;
    int* my = s_cnt + w * nbins;

    // pass 1: count and rank inside the slice
    int kreg[kBucketKeyRegs], rreg[kBucketKeyRegs];
#pragma unroll
    for (int i = 0; i < kBucketKeyRegs; ++i) { kreg[i] = -1; rreg[i] = 0; }
    for (int s0 = t0; s0 < t1; s0 += 32 * kBucketKeyRegs) {
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            const int t = s0 + i * 32 + lane;
            kreg[i] = t < t1 ? __ldg(keys + t) : -1;
        }
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            if (s0 + i * 32 >= t1) break;
            const int k = kreg[i];
            const bool in = k >= 0 && k < nbins;
            const unsigned peers = peers_by_ballot(in, k, bin_bits);
            const int leader = in ? __ffs(peers) - 1 : lane;
            int seen = 0;
            if (in && lane == leader) {
                seen = my[k];
                my[k] = seen + __popc(peers);
            }
            seen = __shfl_sync(kFullMask, seen, leader) + __popc(peers & lt_mask);
            if (in_regs) rreg[i] = seen;
            else if (in) rank_tmp[s0 + i * 32 + lane] = seen;
            __syncwarp();
        }
    }
    __syncthreads();

    // per bin: offsets of the warps inside this CTA; the CTA total goes to row c of the matrix
    for (int b = tid; b < nbins; b += kCoopThreads) {
        int run = 0;
        for (int ww = 0; ww < kCoopWarps; ++ww) {
            const int c2 = s_cnt[ww * nbins + b];
            s_cnt[ww * nbins + b] = run;
            run += c2;
        }
        matrix[c * nbins + b] = run;
    }
    __threadfence();
    cg::this_grid().sync();

    // tokens of the CTAs before this one, and bin totals: column sums of the matrix.  Four bins go in
    // one 16-byte load when nbins % 4 == 0; P threads share a column (P = threads / columns when that is
    // > 1) and every thread keeps kInFlight independent loads in flight.
    if ((nbins & 3) == 0) {
        constexpr int kInFlight = 10;
        const int V = nbins >> 2;
        const int cols = V < kCoopThreads ? V : kCoopThreads;
        const int P = V < kCoopThreads ? kCoopThreads / V : 1;
        const int part = V < kCoopThreads ? tid / V : 0;
        const int4* m4 = reinterpret_cast<const int4*>(matrix);
        for (int vb = tid % cols; vb < V && part < P; vb += kCoopThreads) {
            int4 before = make_int4(0, 0, 0, 0), total = make_int4(0, 0, 0, 0);
            for (int r0 = part; r0 < G; r0 += kInFlight * P) {
                int4 v[kInFlight];
#pragma unroll
                for (int j = 0; j < kInFlight; ++j) {
                    const int r = r0 + j * P;
                    v[j] = r < G ? __ldcg(m4 + r * V + vb) : make_int4(0, 0, 0, 0);
                }
#pragma unroll
                for (int j = 0; j < kInFlight; ++j) {
                    total.x += v[j].x; total.y += v[j].y; total.z += v[j].z; total.w += v[j].w;
                    if (r0 + j * P < c) { before.x += v[j].x; before.y += v[j].y; before.z += v[j].z; before.w += v[j].w; }
                }
            }
            const int b = 4 * vb;
            if (P > 1) {
                atomicAdd(&s_total[b], total.x); atomicAdd(&s_total[b + 1], total.y);
                atomicAdd(&s_total[b + 2], total.z); atomicAdd(&s_total[b + 3], total.w);
                atomicAdd(&s_start[b], before.x); atomicAdd(&s_start[b + 1], before.y);
                atomicAdd(&s_start[b + 2], before.z); atomicAdd(&s_start[b + 3], before.w);
            } else {
                s_total[b] = total.x; s_total[b + 1] = total.y; s_total[b + 2] = total.z; s_total[b + 3] = total.w;
                s_start[b] = before.x; s_start[b + 1] = before.y; s_start[b + 2] = before.z; s_start[b + 3] = before.w;
            }
        }
    } else {
        const int P = nbins < kCoopThreads ? kCoopThreads / nbins : 1;
        for (int b = tid % (nbins < kCoopThreads ? nbins : kCoopThreads); b < nbins; b += kCoopThreads) {
            const int part = nbins < kCoopThreads ? tid / nbins : 0;
            if (part >= P) break;
            int before = 0, total = 0;
            for (int r0 = part; r0 < G; r0 += 8 * P) {
                int v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int r = r0 + j * P;
                    v[j] = r < G ? __ldcg(matrix + r * nbins + b) : 0;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    total += v[j];
                    if (r0 + j * P < c) before += v[j];
                }
            }
            if (P > 1) {
                atomicAdd(&s_total[b], total);
                atomicAdd(&s_start[b], before);
            } else {
                s_total[b] = total;
                s_start[b] = before;      // completed below with the first position of the bin
            }
        }
    }
    __syncthreads();
    // exclusive scan of the totals over the bins (chunks of kCoopThreads bins, running carry)
    int carry = 0;
    for (int b0 = 0; b0 < nbins; b0 += kCoopThreads) {
        const int b = b0 + tid;
        const int v = b < nbins ? s_total[b] : 0;
        int chunk_total = 0;
        const int ex = carry + block_exclusive_scan_nw<kCoopWarps>(v, s_warp, &chunk_total);
        if (b < nbins) {
            const int add = ex + s_start[b];
            for (int ww = 0; ww < kCoopWarps; ++ww) s_cnt[ww * nbins + b] += add;
            s_start[b] = ex;
            if (c == 0) {
                offsets_out[b] = ex;
                if (b == nbins - 1) offsets_out[nbins] = ex + v;
            }
        }
        carry += chunk_total;
    }
    __syncthreads();
    if (tile_rows > 0 && c == 0) {
        int tile_base = 0;
        for (int b0 = 0; b0 < nbins; b0 += kCoopThreads) {
            const int b = b0 + tid;
            const int total = b < nbins ? s_total[b] : 0;
            const int nt = (total + tile_rows - 1) / tile_rows;
            int n_chunk = 0;
            const int tl0 = tile_base + block_exclusive_scan_nw<kCoopWarps>(nt, s_warp, &n_chunk);
            for (int i = 0; i < nt; ++i) {
                Tile tl;
                tl.bin = b;
                tl.start = s_start[b] + i * tile_rows;
                tl.rows = min(tile_rows, total - i * tile_rows);
                tl.pad = 0;
                tiles[tl0 + i] = tl;
            }
            tile_base += n_chunk;
        }
        Tile empty;
        empty.bin = 0; empty.start = 0; empty.rows = 0; empty.pad = 0;
        for (int i = tile_base + tid; i < n_tiles_total; i += kCoopThreads) tiles[i] = empty;
    }

    // pass 2: place
    if (in_regs) {
#pragma unroll
        for (int i = 0; i < kBucketKeyRegs; ++i) {
            const int k = kreg[i];
            if (k >= 0 && k < nbins) perm_out[my[k] + rreg[i]] = t0 + i * 32 + lane;
        }
    } else {
        for (int t = t0 + lane; t < t1; t += 32) {
            const int k = __ldg(keys + t);
            if (k >= 0 && k < nbins) perm_out[my[k] + rank_tmp[t]] = t;
        }
    }
}

// ---- bucketing from per-tile ranks and counts --------------------------------------------------------
// The first descent stage already has every token's key in a register, 128 consecutive tokens per tile.
// It leaves, besides the keys, rank8[t] = number of earlier tokens of t's own tile with the same key, and
// counts8[tile][bin] = tokens of the tile with that key (both fit a byte).  What remains of the stable
// counting sort is then a sum over tiles and a scatter, with no barrier across CTAs: CTA c takes a
// contiguous range of tiles, adds up the counts of all tiles (bin totals) and of the tiles before its
// own (its starting position inside every bin), scans the totals, and places its tokens at
//     start[bin] + tokens of the bin in earlier tiles + rank8[t].
// Every CTA needs those sums over all tiles, so reading the byte matrix row by row made 148 CTAs pull the
// whole matrix through L2 each (6 of the kernel's 8 microseconds at 394 tiles x 256 bins).  The descent
// kernel therefore also adds every tile's counts to block_sums[tile / kRankBlock][bin] (int32 atomics), and a
// CTA here reads that table plus the few byte rows between the last block boundary and its first tile.  The
// table must be zero when the descent kernel starts: the last CTA of this kernel to have read it clears it
// (`done` counts the CTAs; zero before and after every launch).
// Same result as the other bucketing kernels.  Needs 16 <= nbins <= 256 (a multiple of 16) and at most
// kRankedMaxTilesPerCta tiles per CTA.
constexpr int kRankTile = 128;
constexpr int kRankedThreads = 256;
constexpr int kRankedWarps = kRankedThreads / 32;
constexpr int kRankedMaxTilesPerCta = 8;
constexpr int kRankBlock = 16;             // tiles per row of the block-sum table

// The work of one CTA (c of G) of that bucketing, callable from a kernel of its own or as the prologue of a
// larger one: the first kRankedThreads threads of the CTA work, all its threads must call.
// s_dyn: (3 + kRankedMaxTilesPerCta) * nbins ints of shared memory, s_warp: 32 ints.
__device__ __forceinline__ void bucket_ranked_cta(const int32_t* __restrict__ keys, const uint8_t* __restrict__ rank8,
                                                  const uint8_t* __restrict__ counts8, int32_t* block_sums, int* done,
                                                  int32_t* offsets_out, int32_t* perm_out, int B, int nbins, int tile_rows,
                                                  Tile* tiles, int n_tiles_total, int* s_dyn, int* s_warp, int G, int c)
{
    int* s_total = s_dyn;                     // [nbins] tokens in the bin
    int* s_before = s_total + nbins;          // [nbins] of which in tiles before this CTA's
    int* s_start = s_before + nbins;          // [nbins] first position of the bin
    int* s_tile = s_start + nbins;            // [own tiles][nbins] position of the tile's first token of the bin
    const int tid = threadIdx.x;
    const bool on = tid < kRankedThreads;                  // a larger CTA may call this: its other threads only join the barriers
    const int n_src = (B + kRankTile - 1) / kRankTile;
    const int t0 = (int)((int64_t)c * n_src / G), t1 = (int)((int64_t)(c + 1) * n_src / G);

    if (on)
        for (int i = tid; i < 2 * nbins; i += kRankedThreads) s_dyn[i] = 0;
    __syncthreads();

    // everything this thread will need later is requested now, so that the L2 round trips overlap:
    // its tokens' keys and ranks, and (thread = bin) the counts of the CTA's own tiles
    constexpr int kTok = kRankedMaxTilesPerCta * kRankTile / kRankedThreads;
    const int64_t first = (int64_t)t0 * kRankTile, last = min((int64_t)t1 * kRankTile, (int64_t)B);
    int my_key[kTok];
    int my_rank[kTok];
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
        const int64_t t = first + tid + i * kRankedThreads;
        my_key[i] = on && t < last ? __ldg(keys + t) : -1;
        my_rank[i] = on && t < last ? (int)rank8[t] : 0;
    }
    int own[kRankedMaxTilesPerCta];
#pragma unroll
    for (int i = 0; i < kRankedMaxTilesPerCta; ++i)
        own[i] = (tid < nbins && t0 + i < t1) ? (int)counts8[(int64_t)(t0 + i) * nbins + tid] : 0;

    // Column sums of the count matrix.  Whole blocks of kRankBlock tiles come from the block-sum table the descent
    // kernel accumulated (4 bins per 16-byte load), the tiles between the last block boundary and this CTA's first
    // tile from the byte matrix (16 bins per load): one round of loads instead of a pass over every tile's row.
    __shared__ int s_last;
    {
        const int nb = (n_src + kRankBlock - 1) / kRankBlock;
        const int bb = t0 / kRankBlock;                   // blocks that lie entirely before this CTA's tiles
        const int V4 = nbins >> 2;                        // 16-byte columns of the table
        const int P = kRankedThreads / V4;                // threads per column
        const int vb = tid % V4, part = tid / V4;
        const int4* m4 = reinterpret_cast<const int4*>(block_sums);
        int4 tot = make_int4(0, 0, 0, 0), bef = make_int4(0, 0, 0, 0);
        for (int r = part; on && part < P && r < nb; r += 8 * P) {
            int4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = r + j * P < nb ? __ldcg(m4 + (int64_t)(r + j * P) * V4 + vb) : make_int4(0, 0, 0, 0);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                tot.x += v[j].x; tot.y += v[j].y; tot.z += v[j].z; tot.w += v[j].w;
                if (r + j * P < bb) { bef.x += v[j].x; bef.y += v[j].y; bef.z += v[j].z; bef.w += v[j].w; }
            }
        }
        // (the byte row of a tile: nbins / 16 loads; at most kRankBlock - 1 such rows, one load per thread)
        const int V = nbins >> 4;
        const int prow = bb * kRankBlock + tid / V;
        uint4 pv = make_uint4(0, 0, 0, 0);
        const bool partial = on && prow < t0;
        if (partial) pv = __ldcg(reinterpret_cast<const uint4*>(counts8) + (int64_t)prow * V + tid % V);
        if (on && part < P) {
            const int b = 4 * vb;
            if (tot.x) atomicAdd(&s_total[b], tot.x);
            if (tot.y) atomicAdd(&s_total[b + 1], tot.y);
            if (tot.z) atomicAdd(&s_total[b + 2], tot.z);
            if (tot.w) atomicAdd(&s_total[b + 3], tot.w);
            if (bef.x) atomicAdd(&s_before[b], bef.x);
            if (bef.y) atomicAdd(&s_before[b + 1], bef.y);
            if (bef.z) atomicAdd(&s_before[b + 2], bef.z);
            if (bef.w) atomicAdd(&s_before[b + 3], bef.w);
        }
        if (partial) {
            const uint32_t w[4] = {pv.x, pv.y, pv.z, pv.w};
            const int b = 16 * (tid % V);
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int cnt = (int)((w[q] >> (8 * e)) & 0xFFu);
                    if (cnt) atomicAdd(&s_before[b + 4 * q + e], cnt);
                }
        }
    }
    __syncthreads();
    // The table has served this CTA (its values have been used above).  The last CTA to get here clears it for the
    // next descent, at the end of the kernel; the ticket is only looked at there, so nobody waits for it now.
    int ticket = -1;
    if (tid == 0) ticket = atomicAdd(done, 1);

    // exclusive scan of the totals over the bins (nbins <= kRankedThreads)
    {
        const int v = tid < nbins ? s_total[tid] : 0;
        int all = 0;
        const int ex = block_exclusive_scan_nw<kRankedWarps>(v, s_warp, &all);
        if (tid < nbins) {
            s_start[tid] = ex;
            if (c == 0) {
                offsets_out[tid] = ex;
                if (tid == nbins - 1) offsets_out[nbins] = ex + v;
            }
            // positions of this CTA's tiles inside the bin
            int run = ex + s_before[tid];
#pragma unroll
            for (int i = 0; i < kRankedMaxTilesPerCta; ++i) {
                if (t0 + i < t1) s_tile[i * nbins + tid] = run;
                run += own[i];
            }
        }
    }
    __syncthreads();
    // place
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
        const int64_t t = first + tid + i * kRankedThreads;
        const int k = my_key[i];
        if (t < last && k >= 0 && k < nbins) perm_out[s_tile[(int)((t - first) / kRankTile) * nbins + k] + my_rank[i]] = (int32_t)t;
    }

    // tile list: every CTA knows all totals, so each writes the tiles of its share of the bins (bin % G == c) and
    // of the padding
    if (tile_rows > 0) {
        const int total = tid < nbins ? s_total[tid] : 0;
        const int nt = (total + tile_rows - 1) / tile_rows;
        int n_all = 0;
        const int tl0 = block_exclusive_scan_nw<kRankedWarps>(nt, s_warp, &n_all);
        if (tid < nbins && tid % G == c) {
            for (int i = 0; i < nt; ++i) {
                Tile tl;
                tl.bin = tid;
                tl.start = s_start[tid] + i * tile_rows;
                tl.rows = min(tile_rows, total - i * tile_rows);
                tl.pad = 0;
                tiles[tl0 + i] = tl;
            }
        }
        Tile empty;
        empty.bin = 0; empty.start = 0; empty.rows = 0; empty.pad = 0;
        if (on)
            for (int i = n_all + c * kRankedThreads + tid; i < n_tiles_total; i += G * kRankedThreads) tiles[i] = empty;
    }

    // the last CTA to have read the block-sum table clears it and rearms the counter
    if (tid == 0) s_last = ticket == G - 1 ? 1 : 0;
    __syncthreads();
    if (s_last) {
        const int n = (n_src + kRankBlock - 1) / kRankBlock * nbins;
        for (int i = tid; i < n; i += blockDim.x) block_sums[i] = 0;
        if (tid == 0) *done = 0;
    }
}

// Dynamic shared memory: (3 + kRankedMaxTilesPerCta) * nbins ints.
__global__ void __launch_bounds__(kRankedThreads)
k_bucket_ranked(const int32_t* __restrict__ keys, const uint8_t* __restrict__ rank8, const uint8_t* __restrict__ counts8,
                int32_t* __restrict__ block_sums, int* __restrict__ done,
                int32_t* __restrict__ offsets_out, int32_t* __restrict__ perm_out, int B, int nbins, int tile_rows,
                Tile* __restrict__ tiles, int n_tiles_total)
{
    extern __shared__ int s_dyn[];
    __shared__ int s_warp[32];
    pdl_trigger();
    pdl_wait();
    bucket_ranked_cta(keys, rank8, counts8, block_sums, done, offsets_out, perm_out, B, nbins, tile_rows, tiles, n_tiles_total,
                      s_dyn, s_warp,
                      (int)gridDim.x, (int)blockIdx.x);
}

// Tile list from an existing offsets array (one CTA; used when the caller supplies the bucketing),
// padded with empty tiles up to n_tiles_total = floor(B / tile_rows) + nbins.
__global__ void __launch_bounds__(kBucketThreads)
k_tiles_from_offsets(const int32_t* __restrict__ offsets, int nbins, int tile_rows, Tile* __restrict__ tiles,
                     int n_tiles_total)
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
    Tile empty;
    empty.bin = 0; empty.start = 0; empty.rows = 0; empty.pad = 0;
    for (int i = tile_base + threadIdx.x; i < n_tiles_total; i += kBucketThreads) tiles[i] = empty;
}

}  // namespace fff
