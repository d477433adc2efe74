// First stage of the tree descent on the fifth-generation tensor cores (tcgen05, bf16 -> float32).
//
// Algorithm 1, FORWARD_I, non-leaf branch.  At the root every token faces the same subtree, so the
// logits of all 2^k - 1 nodes of its first k <= 8 levels are one dense GEMM
//     logits[B, NP] = X . Wsub^T,        NP = 32, 64, 128 or 256 >= 2^k - 1,
// and the k decisions of a token are read off its row of logits: p <- 2p + 1 + (logit[p] + b[p] >= 0),
// starting at p = 0 in the subtree's breadth-first numbering.  A logit of exactly zero (either sign)
// goes right, NaN goes left, as in the scalar walk.
//
// One persistent CTA per SM works on tiles of 128 consecutive tokens:
//   warp 4   producer: per K-block of 64 columns, one tiled tensor-map load of the 128 x 64 token
//            tile (128-byte swizzled by the copy engine) and one bulk copy of the matching NP x 64
//            slice of the pre-swizzled weight image into a ring of shared-memory stages;
//   warp 5   MMA issuer: four tcgen05.mma (M = 128, N = NP, K = 16) per stage into one of two
//            accumulators in tensor memory; tcgen05.commit frees the stage and, after the last
//            K-block, publishes the accumulator;
//   warps 0-3  epilogue: each thread owns one token (= one tensor-memory lane), reads its NP logits
//            with tcgen05.ld, turns them into NP decision bits, frees the accumulator and walks the
//            subtree on the bits.
// The tensor pipe, the copy engine and the epilogue overlap across tiles through the two accumulators.
//
// The epilogue can also prepare the bucketing by the position just computed (k_bucket_ranked): with the
// 128 keys of a tile in registers, the rank of every token among the equal keys of its tile and the tile's
// count per key cost a few ballots and one pass over a 1 KB table in shared memory.
//
// Every wait is bounded (see ptx.cuh); tensor memory is released on every exit path.
//
// Requirements: bf16, D % 64 == 0, x 16-byte aligned.
#pragma once

#include <cuda.h>      // CUtensorMap

#include "bucket.cuh"
#include "common.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kUM = 128;                 // token rows per tile = rows of one tcgen05.mma
constexpr int kUKB = 64;                 // columns per K-block: 128 bytes, one swizzle line
constexpr int kUmmaEpilogueWarps = 4;
constexpr int kUmmaThreads = (kUmmaEpilogueWarps + 2) * 32;
constexpr int kUmmaMaxStages = 8;

// Decision bits of one token: bit p of bits[] says whether logit[p] + bias[p] >= 0 (a logit of zero goes right,
// NaN left).  The NP logits are this thread's tensor-memory lane, read 32 columns at a time with the next load
// already in flight.
template <int NP>
__device__ __forceinline__ void umma_decision_bits(uint32_t taddr, const float* __restrict__ bias, uint32_t (&bits)[NP / 32])
{
    uint32_t v[2][32];
    ptx::tmem_ld32(taddr, v[0]);
#pragma unroll
    for (int c = 0; c < NP / 32; ++c) {
        ptx::tmem_ld_wait();
        if (c + 1 < NP / 32) ptx::tmem_ld32(taddr + (c + 1) * 32, v[(c + 1) & 1]);
        uint32_t m = 0;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            const float4 b = *reinterpret_cast<const float4*>(bias + c * 32 + j);     // same address in every lane
            m |= (__uint_as_float(v[c & 1][j]) + b.x >= 0.0f ? 1u : 0u) << j;
            m |= (__uint_as_float(v[c & 1][j + 1]) + b.y >= 0.0f ? 1u : 0u) << (j + 1);
            m |= (__uint_as_float(v[c & 1][j + 2]) + b.z >= 0.0f ? 1u : 0u) << (j + 2);
            m |= (__uint_as_float(v[c & 1][j + 3]) + b.w >= 0.0f ? 1u : 0u) << (j + 3);
        }
        bits[c] = m;
    }
}

// The walk p <- 2p + 1 + bit[p] over k levels, p in the subtree's breadth-first numbering.  Level r lives at
// positions 2^r - 1 .. 2^(r+1) - 2, i.e. in words (2^r - 1) / 32 .. (2^(r+1) - 2) / 32 only, so the word is picked
// with as few selects as the level needs (none up to level 4).
template <int NP>
__device__ __forceinline__ int umma_walk(const uint32_t (&bits)[NP / 32], int k)
{
    int p = 0;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        if (r < k && ((1 << r) - 1) < NP) {
            constexpr int kWords = NP / 32;
            const int w_lo = ((1 << r) - 1) >> 5;
            const int w_hi = min(((2 << r) - 2) >> 5, kWords - 1);
            uint32_t w = bits[w_lo < kWords ? w_lo : 0];
#pragma unroll
            for (int c = 1; c < kWords; ++c)
                if (c > w_lo && c <= w_hi) w = (p >> 5) == c ? bits[c] : w;
            p = 2 * p + 1 + (int)((w >> (p & 31)) & 1u);
        }
    }
    return p;
}

// Direct slotting by the position just computed, for a leaf kernel that follows at once: the tokens of a warp
// that reached the same key reserve a run of entries of that key's list with one atomic add on its cursor and
// write their token numbers there: slots[key * cap + cursor .. ), cap >= B.  The order of a list depends on the
// order in which warps arrive, which is harmless for the leaf kernel (the rows of a tile are independent: a
// token's output does not depend on its neighbours) but is not the stable order of the bucketing, so no
// permutation is reported from these lists.  cursor[] is zero on entry and holds the counts per key afterwards.
__device__ __forceinline__ void slot_tokens(bool in, int key, int nbits, int tok, int32_t* __restrict__ cursor,
                                            int32_t* __restrict__ slots, int cap)
{
    const int lane = threadIdx.x & 31;
    const unsigned peers = peers_by_ballot(in, key, nbits);
    const int leader = in ? __ffs(peers) - 1 : lane;
    int base = 0;
    if (in && lane == leader) base = atomicAdd(cursor + key, __popc(peers));
    base = __shfl_sync(kFullMask, base, leader);
    if (in) slots[(int64_t)key * cap + base + __popc(peers & ((1u << lane) - 1u))] = tok;
}

template <int NP> struct DescentUmmaLayout {
    static_assert(NP == 32 || NP == 64 || NP == 128 || NP == 256, "accumulator width");
    static constexpr int kXStageBytes = kUM * kUKB * 2;
    static constexpr int kWStageBytes = NP * kUKB * 2;
    static constexpr int kStageBytes = kXStageBytes + kWStageBytes;          // a multiple of 1024
    static constexpr int kBarrierBytes = 256;                                // 2 * kUmmaMaxStages + 4 mbarriers, tmem slot
    static constexpr int kTmemCols = 2 * NP;                                 // two accumulators
    static constexpr int kCountBytes = kUmmaEpilogueWarps * 256;              // per-warp counts of up to 256 keys, one byte each
    static constexpr int smem_bytes(int stages) { return 1024 + stages * kStageBytes + kBarrierBytes + NP * 4 + kCountBytes; }
};

// wimg: [D / 64][NP rows][64 columns] 128-byte swizzled (the single-group image of k_pack_nodes),
// bimg: [NP] float32.  pos_out[t] = position reached at level k.
// rank8 / counts8 (both or neither, k >= 4): rank8[t] = earlier tokens of t's 128-token tile at the same
// position, counts8[tile][2^k] = tokens of the tile per position.  block_sums (optional, with them):
// [ceil(tiles / kRankBlock)][2^k] int32, zero on entry, to which the counts of every block of kRankBlock
// consecutive tiles are added (integer atomics: the sums do not depend on the order).
// pos_out2 (optional): a second copy of the positions.  cursor / slots / cap (optional, instead of the ranks):
// see slot_tokens.
template <int NP>
__global__ void __launch_bounds__(kUmmaThreads, 1)
k_descent_umma(const __grid_constant__ CUtensorMap tmap_x, const __nv_bfloat16* __restrict__ wimg,
               const float* __restrict__ bimg, int32_t* __restrict__ pos_out, uint8_t* __restrict__ rank8,
               uint8_t* __restrict__ counts8, int32_t* __restrict__ block_sums, int32_t* __restrict__ pos_out2,
               int32_t* __restrict__ cursor, int32_t* __restrict__ slots, int cap, int D, int B, int k, int kStages,
               int* __restrict__ status)
{
    using L = DescentUmmaLayout<NP>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(ring + kStages * L::kStageBytes);
    uint64_t* empty = full + kUmmaMaxStages;
    uint64_t* acc_full = empty + kUmmaMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    float* bias = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(full) + L::kBarrierBytes);
    uint8_t* s_cnt = reinterpret_cast<uint8_t*>(bias + NP);                   // [epilogue warp][256]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = (B + kUM - 1) / kUM;
    const int KB = D / kUKB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, 1);
            ptx::mbar_init(empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full + a, 1);
            ptx::mbar_init(acc_empty + a, kUmmaEpilogueWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    if (warp == 5) {
        ptx::tmem_alloc(tmem_slot, L::kTmemCols);
        ptx::tmem_relinquish_alloc_permit();
    }
    for (int i = threadIdx.x; i < NP; i += kUmmaThreads) bias[i] = bimg[i];    // a parameter image, not a predecessor's output
    for (int i = threadIdx.x; i < L::kCountBytes / 4; i += kUmmaThreads) reinterpret_cast<uint32_t*>(s_cnt)[i] = 0;
    ptx::tc_fence_before_sync();
    pdl_trigger();
    __syncthreads();
    ptx::tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = *tmem_slot;

    bool timed_out = false;
    if (warp == 4) {
        // ------------------------------------------------------------------ producer
        int stage = 0;
        uint32_t phase = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                if (lane == 0) {
                    unsigned char* st = ring + stage * L::kStageBytes;
                    ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)L::kStageBytes);
                    ptx::tma_load_2d(st, &tmap_x, kb * kUKB, tile * kUM, full + stage);
                    ptx::bulk_g2s(st + L::kXStageBytes, wimg + (int64_t)kb * (NP * kUKB), L::kWStageBytes, full + stage);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(kUM, NP);
        int stage = 0;
        uint32_t phase = 0;
        int it = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int a = it & 1;
            if (!timed_out && !ptx::mbar_wait(acc_empty + a, ((it >> 1) & 1) ^ 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t xs = ptx::smem_addr(ring + stage * L::kStageBytes);
                    const uint64_t ad = ptx::umma_desc_k128(xs), bd = ptx::umma_desc_k128(xs + L::kXStageBytes);
#pragma unroll
                    for (int j = 0; j < kUKB / 16; ++j)
                        ptx::umma_bf16(tmem_base + a * NP, ad + 2 * j, bd + 2 * j, idesc, (kb | j) != 0 ? 1u : 0u);
                    ptx::umma_commit(empty + stage);
                    if (kb == KB - 1) ptx::umma_commit(acc_full + a);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token per thread
        // Pass -1 is a rehearsal: while the first accumulator is still being computed, the warps run once through the
        // epilogue's code on whatever tensor memory holds, with every wait, store and atomic switched off.  A launch
        // starts with a cold instruction cache, and the first real pass took ten times as long as the later ones
        // (measured: 11.6 us against 1.1 us per tile).  Where the loads run ahead anyway (64 nodes, 1024 inputs) that
        // hid behind them; with 256 nodes on single CTAs it was exposed (first stage of a 15-level tree: 18.4 -> 17.1 us).
        for (int it = -1, tile = blockIdx.x; tile < n_tiles; ++it, tile += it > 0 ? gridDim.x : 0) {
            const bool dry = it < 0;
            const int a = it & 1;
            if (!dry && !timed_out && !ptx::mbar_wait(acc_full + a, (it >> 1) & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            uint32_t bits[NP / 32];
            umma_decision_bits<NP>(tmem_base + ((uint32_t)(warp * 32) << 16) + a * NP, bias, bits);
            ptx::tc_fence_before_sync();
            if (!dry) ptx::mbar_arrive(acc_empty + a);

            const int p = umma_walk<NP>(bits, k);
            const int tok = tile * kUM + warp * 32 + lane;
            const int key = p - ((1 << k) - 1);
            const bool in = !dry && tok < B;
            if (in) {
                pos_out[tok] = key;
                if (pos_out2) pos_out2[tok] = key;
            }
            if (cursor) {
                slot_tokens(in, key, k, tok, cursor, slots, cap);
            } else if (rank8) {
                const int nbins = 1 << k;
                const unsigned peers = peers_by_ballot(in, key, k);
                if (in && lane == __ffs(peers) - 1) s_cnt[warp * 256 + key] = (uint8_t)__popc(peers);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (in) {
                    int before = __popc(peers & ((1u << lane) - 1u));
                    for (int w = 0; w < warp; ++w) before += s_cnt[w * 256 + key];
                    rank8[tok] = (uint8_t)before;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                for (int b = warp * 32 + lane; b < nbins; b += kUmmaEpilogueWarps * 32) {
                    int total = 0;
#pragma unroll
                    for (int w = 0; w < kUmmaEpilogueWarps; ++w) {
                        total += s_cnt[w * 256 + b];
                        s_cnt[w * 256 + b] = 0;
                    }
                    if (!dry) counts8[(int64_t)tile * nbins + b] = (uint8_t)total;
                    if (block_sums && total > 0) atomicAdd(block_sums + (int64_t)(tile / kRankBlock) * nbins + b, total);
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let copies and MMAs still in flight finish before exit
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, L::kTmemCols);
    }
}

// ---- the first stage on CTA pairs ----------------------------------------------------------------------
// With NP = 128 or 256 the weight K-blocks (16-32 KB each) are re-streamed from L2 for every 128-token tile,
// and that traffic, not DRAM, bounds the kernel above.  Here two CTAs (a cluster of two, cta_group::2) share
// every weight K-block: each loads its own 128-token tile of x and HALF of the NP weight rows, the pair's first
// CTA issues one MMA over 256 rows that reads A and B from both CTAs' shared memory, and each CTA keeps the
// accumulator rows of its own tokens in its own tensor memory.  Roles per CTA as above; differences:
//   * the "stage full" and "accumulator free" barriers that the MMA issuer waits on live in the first CTA; the
//     second CTA's producer and epilogue arrive on them through the shared::cluster window, and its tensor-map
//     loads (cta_group::2 form) count their bytes there;
//   * tcgen05.commit frees a stage / publishes an accumulator in both CTAs (one commit per CTA);
//   * the weight image is read through a tensor map of its own (rows of 64 columns, no swizzle mode: the image
//     is stored pre-swizzled), because only tensor-map loads can signal the other CTA's barrier;
//   * cluster barriers order barrier initialisation before the first remote arrival, and the last remote
//     operation before either CTA leaves.
template <int NP> struct DescentUmmaPairLayout {
    static_assert(NP == 128 || NP == 256, "accumulator width");
    static constexpr int kXStageBytes = kUM * kUKB * 2;
    static constexpr int kWStageBytes = (NP / 2) * kUKB * 2;                 // this CTA's half of the weight rows
    static constexpr int kStageBytes = kXStageBytes + kWStageBytes;          // a multiple of 1024
    static constexpr int kBarrierBytes = 256;
    static constexpr int kTmemCols = 2 * NP;                                 // two accumulators (per CTA)
    static constexpr int kCountBytes = kUmmaEpilogueWarps * 256;
    static constexpr int smem_bytes(int stages) { return 1024 + stages * kStageBytes + kBarrierBytes + NP * 4 + kCountBytes; }
};

// tmap_w: the single-group image as a matrix of (D/64) * NP rows of 64 columns, boxes of NP/2 rows.
template <int NP>
__global__ void __launch_bounds__(kUmmaThreads, 1)
k_descent_umma_pair(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    const float* __restrict__ bimg, int32_t* __restrict__ pos_out, uint8_t* __restrict__ rank8,
                    uint8_t* __restrict__ counts8, int32_t* __restrict__ block_sums, int32_t* __restrict__ pos_out2,
                    int32_t* __restrict__ cursor, int32_t* __restrict__ slots, int cap, int D, int B, int k, int kStages,
                    int* __restrict__ status)
{
    namespace cg = cooperative_groups;
    using L = DescentUmmaPairLayout<NP>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(ring + kStages * L::kStageBytes);     // used in the first CTA only
    uint64_t* empty = full + kUmmaMaxStages;
    uint64_t* acc_full = empty + kUmmaMaxStages;
    uint64_t* acc_empty = acc_full + 2;                                                 // used in the first CTA only
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    float* bias = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(full) + L::kBarrierBytes);
    uint8_t* s_cnt = reinterpret_cast<uint8_t*>(bias + NP);

    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();            // 0: issues the MMAs
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = (B + kUM - 1) / kUM;
    const int n_pairs = (n_tiles + 1) / 2;
    const int pair0 = blockIdx.x >> 1, pair_stride = gridDim.x >> 1;
    const int KB = D / kUKB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, 2);                   // one arrival (with its byte count) per CTA
            ptx::mbar_init(empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full + a, 1);
            ptx::mbar_init(acc_empty + a, 2 * kUmmaEpilogueWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
        ptx::prefetch_tensormap(&tmap_w);
    }
    if (warp == 5) {
        ptx::tmem_alloc_pair(tmem_slot, L::kTmemCols);
        ptx::tmem_relinquish_alloc_permit_pair();
    }
    for (int i = threadIdx.x; i < NP; i += kUmmaThreads) bias[i] = bimg[i];
    for (int i = threadIdx.x; i < L::kCountBytes / 4; i += kUmmaThreads) reinterpret_cast<uint32_t*>(s_cnt)[i] = 0;
    ptx::tc_fence_before_sync();
    pdl_trigger();
    cluster.sync();                                        // both CTAs' barriers exist before anything arrives on them
    ptx::tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = *tmem_slot;

    bool timed_out = false;
    if (warp == 4) {
        // ------------------------------------------------------------------ producer (each CTA: its tile, its half of W)
        int stage = 0;
        uint32_t phase = 0;
        for (int pair = pair0; pair < n_pairs; pair += pair_stride) {
            const int tile = 2 * pair + (int)rank;         // may be one past the end: such rows read as zeros
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                if (lane == 0) {
                    unsigned char* st = ring + stage * L::kStageBytes;
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_addr(full + stage), 0);
                    ptx::mbar_arrive_expect_tx_cluster(bar, (uint32_t)L::kStageBytes);
                    ptx::tma_load_2d_pair(st, &tmap_x, kb * kUKB, tile * kUM, bar);
                    ptx::tma_load_2d_pair(st + L::kXStageBytes, &tmap_w, 0, kb * NP + (int)rank * (NP / 2), bar);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer (first CTA only)
        if (rank == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(2 * kUM, NP);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            for (int pair = pair0; pair < n_pairs; pair += pair_stride, ++it) {
                const int a = it & 1;
                if (!timed_out && !ptx::mbar_wait(acc_empty + a, ((it >> 1) & 1) ^ 1)) timed_out = true;
                ptx::tc_fence_after_sync();
                for (int kb = 0; kb < KB; ++kb) {
                    if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                    ptx::tc_fence_after_sync();
                    if (lane == 0) {
                        const uint32_t xs = ptx::smem_addr(ring + stage * L::kStageBytes);
                        const uint64_t ad = ptx::umma_desc_k128(xs), bd = ptx::umma_desc_k128(xs + L::kXStageBytes);
#pragma unroll
                        for (int j = 0; j < kUKB / 16; ++j)
                            ptx::umma_bf16_pair(tmem_base + a * NP, ad + 2 * j, bd + 2 * j, idesc, (kb | j) != 0 ? 1u : 0u);
                        const uint32_t e0 = ptx::smem_addr(empty + stage);
                        ptx::umma_commit_pair(ptx::map_to_cta(e0, 0));
                        ptx::umma_commit_pair(ptx::map_to_cta(e0, 1));
                        if (kb == KB - 1) {
                            const uint32_t f0 = ptx::smem_addr(acc_full + a);
                            ptx::umma_commit_pair(ptx::map_to_cta(f0, 0));
                            ptx::umma_commit_pair(ptx::map_to_cta(f0, 1));
                        }
                    }
                    __syncwarp();
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token per thread
        // (pass -1 is the rehearsal that warms the instruction cache, see k_descent_umma)
        for (int it = -1, pair = pair0; pair < n_pairs; ++it, pair += it > 0 ? pair_stride : 0) {
            const bool dry = it < 0;
            const int tile = 2 * pair + (int)rank;
            const int a = it & 1;
            if (!dry && !timed_out && !ptx::mbar_wait(acc_full + a, (it >> 1) & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            uint32_t bits[NP / 32];
            umma_decision_bits<NP>(tmem_base + ((uint32_t)(warp * 32) << 16) + a * NP, bias, bits);
            ptx::tc_fence_before_sync();
            // (relaxed: the loads above have completed, there is nothing else of this thread to publish)
            if (!dry) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_addr(acc_empty + a), 0));

            const int p = umma_walk<NP>(bits, k);
            const int tok = tile * kUM + warp * 32 + lane;
            const int key = p - ((1 << k) - 1);
            const bool in = !dry && tok < B;
            if (in) {
                pos_out[tok] = key;
                if (pos_out2) pos_out2[tok] = key;
            }
            if (cursor) {
                slot_tokens(in, key, k, tok, cursor, slots, cap);
            } else if (rank8) {
                const int nbins = 1 << k;
                const unsigned peers = peers_by_ballot(in, key, k);
                if (in && lane == __ffs(peers) - 1) s_cnt[warp * 256 + key] = (uint8_t)__popc(peers);
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (in) {
                    int before = __popc(peers & ((1u << lane) - 1u));
                    for (int w = 0; w < warp; ++w) before += s_cnt[w * 256 + key];
                    rank8[tok] = (uint8_t)before;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (!dry && tile < n_tiles) {
                    for (int b = warp * 32 + lane; b < nbins; b += kUmmaEpilogueWarps * 32) {
                        int total = 0;
#pragma unroll
                        for (int w = 0; w < kUmmaEpilogueWarps; ++w) {
                            total += s_cnt[w * 256 + b];
                            s_cnt[w * 256 + b] = 0;
                        }
                        counts8[(int64_t)tile * nbins + b] = (uint8_t)total;
                        if (block_sums && total > 0) atomicAdd(block_sums + (int64_t)(tile / kRankBlock) * nbins + b, total);
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    cluster.sync();                                        // nothing of the pair is in flight any more
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, L::kTmemCols);
    }
}

// ---- later stages: tokens grouped by the node they have reached -------------------------------------
// The same dense evaluation for a stage that starts at level L0 > 0: the tokens have been bucketed by their
// node at level L0 (perm, and a list of tiles of up to 128 consecutive entries of one bucket), every bucket
// has its own subtree image, and the rows of a tile are gathered through the permutation with tile::gather4
// tensor-map loads (4 rows x 128 bytes per request, 128-byte swizzled by the copy engine).
//   warps 0-3  epilogue, as above; pos_out[token] = (node << k) + position inside the subtree;
//   warp 4     MMA issuer;
//   warps 5-8  gathers, the 4-row groups of a tile dealt round-robin to the four warps; the first of them
//              also starts the bulk copy of the bucket's weight K-blocks.
// A ring stage holds two K-blocks of 64 columns.  CTAs walk the tile list with a static stride and skip its
// empty entries; rows of a ragged tile beyond its length are not loaded and their logits never used.
constexpr int kUGGatherWarps = 4;
constexpr int kUGThreads = (kUmmaEpilogueWarps + 1 + kUGGatherWarps) * 32;
constexpr int kUGSub = 2;                                  // K-blocks per ring stage
constexpr int kUGMaxBins = 256;                            // nodes of the first stage's last level (direct lists)

template <int NP> struct DescentUmmaGroupedLayout {
    static_assert(NP == 16 || NP == 32 || NP == 64, "accumulator width");
    static constexpr int kXSubBytes = kUM * kUKB * 2;
    static constexpr int kWSubBytes = NP * kUKB * 2;
    static constexpr int kXStageBytes = kUGSub * kXSubBytes;
    static constexpr int kWStageBytes = kUGSub * kWSubBytes;
    static constexpr int kStageBytes = kXStageBytes + kWStageBytes;          // a multiple of 1024
    static constexpr int kBarrierBytes = 256;
    static constexpr int kTmemCols = 2 * NP < 64 ? 64 : 2 * NP;              // two accumulators; the epilogue always loads 32 columns
    static constexpr int kListBytes = (2 * kUGMaxBins + 1 + 16) * 4;          // direct lists: counts, tile prefix, warp sums
    static constexpr int smem_bytes(int stages) { return 1024 + stages * kStageBytes + kBarrierBytes + 2 * NP * 4 + kListBytes; }
};

// wimg: [group][D / 64][NP rows][64 columns] swizzled, bimg: [group][NP] float32 (k_pack_nodes).
// pos_out2 / cursor / slots / cap (optional): as in the first stage (slot_tokens).
// node_counts (optional, n_bins <= kUGMaxBins): instead of a tile list and a permutation, the lists the first stage
// filled directly (slot_tokens): perm[bin * node_cap + i], i < node_counts[bin], are the tokens that reached node
// `bin`.  Every CTA then derives the tiles itself (tile t of the launch = the (t - tiles before its bin)-th run of
// 128 entries of that bin's list), which saves the node bucketing launch in between.  node_counts[kUGMaxBins] counts
// the CTAs that have finished; the last one clears the counts and that word for the next call.
template <int NP>
__global__ void __launch_bounds__(kUGThreads, 1)
k_descent_umma_grouped(const __grid_constant__ CUtensorMap tmap_x, const int32_t* __restrict__ perm,
                       const Tile* __restrict__ tiles, int n_tiles_total, const __nv_bfloat16* __restrict__ wimg,
                       const float* __restrict__ bimg, int32_t* __restrict__ pos_out, int32_t* __restrict__ pos_out2,
                       int32_t* __restrict__ cursor, int32_t* __restrict__ slots, int cap, int D, int k, int kStages,
                       int* __restrict__ status, int32_t* __restrict__ node_counts, int n_bins, int node_cap)
{
    using L = DescentUmmaGroupedLayout<NP>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(ring + kStages * L::kStageBytes);
    uint64_t* empty = full + kUmmaMaxStages;
    uint64_t* acc_full = empty + kUmmaMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    float* bias = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(full) + L::kBarrierBytes);     // [2][NP]
    int* s_cnt = reinterpret_cast<int*>(bias + 2 * NP);    // [kUGMaxBins] tokens per node (direct lists)
    int* s_tpre = s_cnt + kUGMaxBins;                      // [kUGMaxBins + 1] tiles before each node
    int* s_wsum = s_tpre + kUGMaxBins + 1;                 // [16]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = D / (kUKB * kUGSub);                    // ring stages per tile

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, kUGGatherWarps);      // one arrival per gather warp
            ptx::mbar_init(empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full + a, 1);
            ptx::mbar_init(acc_empty + a, kUmmaEpilogueWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    if (warp == 4) {
        ptx::tmem_alloc(tmem_slot, L::kTmemCols);
        ptx::tmem_relinquish_alloc_permit();
    }
    ptx::tc_fence_before_sync();
    pdl_trigger();
    __syncthreads();
    ptx::tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = *tmem_slot;

    // direct lists: tiles per node and their running sum, by every CTA for itself (n_bins <= 256 <= threads)
    if (node_counts) {
        const int tid = threadIdx.x;
        const int c = tid < n_bins ? node_counts[tid] : 0;
        const int t = (c + kUM - 1) / kUM;
        int incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(kFullMask, incl, o);
            if (lane >= o) incl += v;
        }
        if (tid < kUGMaxBins) s_cnt[tid] = c;
        if (lane == 31) s_wsum[warp] = incl;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < warp; ++w) before += s_wsum[w];
        if (tid < n_bins) s_tpre[tid + 1] = before + incl;
        if (tid == 0) s_tpre[0] = 0;
        __syncthreads();
        n_tiles_total = s_tpre[n_bins];
    }
    // tile `idx` of the launch
    auto tile_at = [&](int idx) {
        if (!node_counts) return tiles[idx];
        int lo = 0, hi = n_bins;                              // s_tpre[lo] <= idx < s_tpre[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_tpre[mid] <= idx) lo = mid;
            else hi = mid;
        }
        const int local = idx - s_tpre[lo];
        Tile tl;
        tl.bin = lo;
        tl.start = lo * node_cap + local * kUM;
        tl.rows = min(kUM, s_cnt[lo] - local * kUM);
        tl.pad = 0;
        return tl;
    };

    bool timed_out = false;
    if (warp > 4) {
        // ------------------------------------------------------------------ row gathers (+ weight copies)
        const int gw = warp - 5;
        int stage = 0;
        uint32_t phase = 0;
        for (int tile = blockIdx.x; tile < n_tiles_total; tile += gridDim.x) {
            const Tile tl = tile_at(tile);
            if (tl.rows <= 0) continue;
            const int total_groups = (tl.rows + 3) >> 2;
            const int groups = max((total_groups - gw + kUGGatherWarps - 1) / kUGGatherWarps, 0);
            const int first = (lane * kUGGatherWarps + gw) * 4;
            int r[4] = {0, 0, 0, 0};
            if (lane < groups) {
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = perm[tl.start + min(first + i, tl.rows - 1)];
            }
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                unsigned char* st = ring + stage * L::kStageBytes;
                if (lane == 0) {
                    const uint32_t bytes = (uint32_t)groups * (512u * kUGSub) + (gw == 0 ? (uint32_t)L::kWStageBytes : 0u);
                    if (bytes > 0) ptx::mbar_arrive_expect_tx(full + stage, bytes);
                    else ptx::mbar_arrive(full + stage);
                    if (gw == 0)
                        ptx::bulk_g2s(st + L::kXStageBytes, wimg + ((int64_t)tl.bin * KB + kb) * (kUGSub * NP * kUKB), L::kWStageBytes,
                                      full + stage);
                }
                __syncwarp();
                if (lane < groups) {
#pragma unroll
                    for (int sb = 0; sb < kUGSub; ++sb)
                        ptx::tma_gather4(st + sb * L::kXSubBytes + first * 128, &tmap_x, (kb * kUGSub + sb) * kUKB, r[0], r[1], r[2], r[3],
                                         full + stage);
                }
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(kUM, NP);
        int stage = 0;
        uint32_t phase = 0;
        int it = 0;
        for (int tile = blockIdx.x; tile < n_tiles_total; tile += gridDim.x) {
            if (tile_at(tile).rows <= 0) continue;
            const int a = it & 1;
            if (!timed_out && !ptx::mbar_wait(acc_empty + a, ((it >> 1) & 1) ^ 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t xs = ptx::smem_addr(ring + stage * L::kStageBytes);
#pragma unroll
                    for (int sb = 0; sb < kUGSub; ++sb) {
                        const uint64_t ad = ptx::umma_desc_k128(xs + sb * L::kXSubBytes);
                        const uint64_t bd = ptx::umma_desc_k128(xs + L::kXStageBytes + sb * L::kWSubBytes);
#pragma unroll
                        for (int j = 0; j < kUKB / 16; ++j)
                            ptx::umma_bf16(tmem_base + a * NP, ad + 2 * j, bd + 2 * j, idesc, (kb | sb | j) != 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(empty + stage);
                    if (kb == KB - 1) ptx::umma_commit(acc_full + a);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
            ++it;
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token per thread
        int it = 0;
        for (int tile = blockIdx.x; tile < n_tiles_total; tile += gridDim.x) {
            const Tile tl = tile_at(tile);
            if (tl.rows <= 0) continue;
            const int a = it & 1;
            const int row = warp * 32 + lane;
            const int64_t tok = row < tl.rows ? perm[tl.start + row] : -1;
            // this bucket's biases; the buffer of two tiles ago is free: its readers have passed the barrier
            // of the previous tile
            float* tb = bias + a * NP;
            if (row < NP) tb[row] = __ldg(bimg + (int64_t)tl.bin * NP + row);
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (!timed_out && !ptx::mbar_wait(acc_full + a, (it >> 1) & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            uint32_t bits = 0, bits_hi = 0;
            {
                uint32_t v[32];
                ptx::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + a * NP, v);      // columns past NP are not used
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32 && j < NP; ++j) bits |= (__uint_as_float(v[j]) + tb[j] >= 0.0f ? 1u : 0u) << j;
                if (NP == 64) {
                    ptx::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + a * NP + 32, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) bits_hi |= (__uint_as_float(v[j]) + tb[32 + j] >= 0.0f ? 1u : 0u) << j;
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(acc_empty + a);
            int p = 0;
            for (int r = 0; r < k; ++r) {
                const uint32_t w = (NP == 64 && p >= 32) ? bits_hi : bits;
                p = 2 * p + 1 + (int)((w >> (p & 31)) & 1u);
            }
            const int key = (tl.bin << k) + (p - ((1 << k) - 1));
            if (tok >= 0) {
                pos_out[tok] = key;
                if (pos_out2) pos_out2[tok] = key;
            }
            // (the keys of a tile differ in their low k bits only)
            if (cursor) slot_tokens(tok >= 0, key, k, (int)tok, cursor, slots, cap);
            ++it;
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let copies and MMAs still in flight finish before exit
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, L::kTmemCols);
    }
    // the last CTA to finish rearms the direct lists' counts (every CTA has read them long ago: before its first tile)
    if (node_counts && warp == 0) {
        int is_last = 0;
        if (lane == 0) {
            __threadfence();
            is_last = atomicAdd(node_counts + kUGMaxBins, 1) == (int)gridDim.x - 1 ? 1 : 0;
        }
        is_last = __shfl_sync(kFullMask, is_last, 0);
        if (is_last) {
            for (int b = lane; b < n_bins; b += 32) node_counts[b] = 0;
            if (lane == 0) node_counts[kUGMaxBins] = 0;
            __threadfence();
        }
    }
}

}  // namespace fff
