// One stage of the tree descent on tensor cores (bf16, float32 accumulate).
//
// Algorithm 1, FORWARD_I, non-leaf branch.  The d sequential node decisions of a token are cut into
// stages of k <= 6 levels.  A stage starts with the tokens grouped by the node they have reached at
// level L0 (all tokens at the root for the first stage).  For one group, the 2^k - 1 nodes of the
// depth-k subtree below that node are the same for every token of the group, so their logits are one
// narrow GEMM,
//     logits[|group|, NP] = X[group] . Wsub^T,        NP = 16, 32 or 64 >= 2^k - 1,
// and the k decisions are then read off the logits by walking the subtree: position p <- 2p + 1 +
// (logit[p] + b[p] >= 0), starting at p = 0 in the subtree's own breadth-first numbering.  This trades
// (2^k - 1) / k times more multiply-adds, which the tensor cores absorb, for k times fewer passes
// over x and no per-token fetch of weight rows.
//
// The machinery is that of the grouped leaf kernel: persistent CTAs over a tile list (tiles of up to
// 64 consecutive entries of one group), producer warps that copy the gathered token rows with
// 16-byte cp.async and a pre-swizzled weight image with one bulk (TMA) copy per stage into an
// mbarrier ring, and 8 consumer warps with mma.sync.m16n8k16 (two per 16-row m-tile, taking alternate
// k-steps).  tiles == NULL means "one group, tokens in natural order".
//
// Requirements: bf16, D % kKS == 0.
#pragma once

#include "common.cuh"
#include "leaf_mma.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kDTM = 64;                                   // token rows per tile of the descent stages
constexpr int kDescentMTiles = kDTM / 16;
// Two warps share each 16-row m-tile and take alternate k-steps (a single warp would crawl along one
// chain of dependent mma); the pair adds its partial logits up through shared memory.
constexpr int kDescentKSplit = 2;
constexpr int kDescentConsumers = kDescentMTiles * kDescentKSplit;
constexpr int kDescentThreads = (kDescentConsumers + kProducerWarps) * 32;

// The ring depth and the stage stride are run-time values: a stage holds the token rows and, unless the
// whole weight image of the (single) group is kept resident in shared memory, the matching weight slice.
template <int NP> struct DescentMmaLayout {
    static constexpr int kWStageBytes = NP * kKS * 2;
    static constexpr int kXStageBytes = kDTM * kXRowBytes;
    static constexpr int kStageBytes = kXStageBytes + kWStageBytes;
    static constexpr int kStageStride = (kStageBytes + 127) & ~127;
    static constexpr int kLogitRow = NP + 1;                                     // floats, padded
    // one scratch area per warp pair: partial accumulators (fragment order), then the 16 logit rows
    static constexpr int kPairScratch = (16 * kLogitRow * 4 > NP * 64 ? 16 * kLogitRow * 4 : NP * 64);
    static constexpr int kStagingBytes = kDescentMTiles * kPairScratch;
    static constexpr int kFixedBytes = ((kStagingBytes + 127) & ~127) + 256 /* barriers */ + 128 /* align */;
    // shared memory of a launch with `stages` ring stages; resident_bytes = NP * D * 2 or 0
    static constexpr int smem_bytes(int stages, int resident_bytes) {
        return stages * (resident_bytes ? kXStageBytes : kStageStride) + kFixedBytes + resident_bytes;
    }
};

// Weight image of one stage: [group][D/kKS][kKS/64][NP rows][64 columns] 128-byte swizzled, rows in the
// subtree's breadth-first order (row 2^r - 1 + p = node N_{L0+r, g*2^r + p}); unused rows zero.
// Bias image: [group][NP] float32.
template <typename T>
__global__ void k_pack_nodes(const T* __restrict__ node_w, const T* __restrict__ node_b,
                             __nv_bfloat16* __restrict__ img, float* __restrict__ bimg,
                             int L0, int k, int NP, int D)
{
    const int64_t groups = (int64_t)1 << L0;
    const int64_t total = groups * NP * D;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int kk = (int)(i % D);
        const int n = (int)((i / D) % NP);
        const int64_t g = i / ((int64_t)D * NP);
        int r = 0;
        while (((1 << (r + 1)) - 1) <= n) ++r;                 // level of local node n inside the subtree
        const bool used = r < k;
        const int64_t p = n - ((1 << r) - 1);
        const int64_t row = used ? (((int64_t)1 << (L0 + r)) - 1 + g * ((int64_t)1 << r) + p) : 0;
        const int u = kk / kKS, sb = (kk % kKS) / 64, kc = kk % 64;
        const uint32_t off = ptx::swz128((uint32_t)((sb * NP + n) * 128 + kc * 2));
        const int64_t base = (g * (D / kKS) + u) * (int64_t)(NP * kKS);
        img[base + off / 2] = __float2bfloat16_rn(used ? Elem<T>::to_float(node_w[row * D + kk]) : 0.0f);
        if (kk == 0) bimg[g * NP + n] = used ? Elem<T>::to_float(node_b[row]) : 0.0f;
    }
}

// resident != 0 (single-group stage only, tiles == NULL): the whole weight image of the group is copied
// into shared memory once per CTA and the ring carries token rows only.
template <int NP>
__global__ void __launch_bounds__(kDescentThreads, NP <= 32 ? 2 : 1)
k_descent_mma(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ perm,
              const Tile* __restrict__ tiles, int n_tiles_total,
              const __nv_bfloat16* __restrict__ wimg, const float* __restrict__ bimg,
              int32_t* __restrict__ pos_out,
              int D, int B, int k, int kStages, int resident, int* __restrict__ status)
{
    using L = DescentMmaLayout<NP>;
    constexpr int kTM = kDTM;
    constexpr int kLeafMmaConsumers = kDescentConsumers;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int stage_stride = resident ? L::kXStageBytes : L::kStageStride;
    unsigned char* stages = smem;
    unsigned char* staging = smem + kStages * stage_stride;
    uint64_t* full = reinterpret_cast<uint64_t*>(staging + ((L::kStagingBytes + 127) & ~127));
    uint64_t* empty = full + kMaxStages;
    uint64_t* wbar = empty + kMaxStages;                               // completion of the resident weight copy
    unsigned char* wres = reinterpret_cast<unsigned char*>(full) + 256;  // resident weight image

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int U1 = D / kKS;
    const int ntiles = n_tiles_total;      // a device-built list may contain empty tiles (rows = 0)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, kProducerThreads + 1);     // every producer thread + the weight copy
            ptx::mbar_init(empty + s, kLeafMmaConsumers);
        }
        ptx::mbar_init(wbar, 1);
        ptx::fence_mbar_init();
    }
    pdl_trigger();
    __syncthreads();
    pdl_wait();
    if (resident && threadIdx.x == 0) {
        ptx::mbar_arrive_expect_tx(wbar, (uint32_t)(NP * D * 2));
        for (int u = 0; u < D / kKS; ++u)
            ptx::bulk_g2s(wres + u * L::kWStageBytes, wimg + (int64_t)u * (NP * kKS), L::kWStageBytes, wbar);
    }

    int stage = 0;
    uint32_t phase = 0;
    bool timed_out = false;

    auto get_tile = [&](int t) {
        Tile tl;
        if (tiles) {
            tl = tiles[t];
        } else {
            tl.bin = 0;
            tl.start = t * kTM;
            tl.rows = min(kTM, B - t * kTM);
            tl.pad = 0;
        }
        return tl;
    };

    if (warp >= kLeafMmaConsumers) {
        // ------------------------------------------------------------------ producer warps
        const int ptid = threadIdx.x - kLeafMmaConsumers * 32;
        const int prow = ptid >> 4, pchunk = ptid & 15;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const Tile tl = get_tile(tile);
            if (tl.rows == 0) continue;
            const __nv_bfloat16* src[kTM / kRowsPerPass];
#pragma unroll
            for (int i = 0; i < kTM / kRowsPerPass; ++i) {
                const int r = i * kRowsPerPass + prow;
                const int64_t tok = r < tl.rows ? (perm ? perm[tl.start + r] : tl.start + r) : -1;
                src[i] = tok >= 0 ? x + tok * D + pchunk * 8 : nullptr;
            }
            for (int u = 0; u < U1; ++u) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                unsigned char* st = stages + stage * stage_stride;
                if (ptid == 0) {
                    if (resident) {
                        ptx::mbar_arrive(full + stage);
                    } else {
                        ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)L::kWStageBytes);
                        ptx::bulk_g2s(st + kTM * kXRowBytes, wimg + ((int64_t)tl.bin * U1 + u) * (NP * kKS), L::kWStageBytes,
                                      full + stage);
                    }
                }
#pragma unroll
                for (int i = 0; i < kTM / kRowsPerPass; ++i)
                    if (src[i]) ptx::cp_async16(st + (i * kRowsPerPass + prow) * kXRowBytes + pchunk * 16, src[i] + u * kKS);
                ptx::cp_async_mbar_arrive(full + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int mi = warp % kDescentMTiles, ni = warp / kDescentMTiles;
        const int m0 = mi * 16;
        float* pair = reinterpret_cast<float*>(staging + mi * L::kPairScratch);
        const int g = lane >> 2, q4 = lane & 3;
        const int bn = (lane & 7) + ((lane >> 4) << 3);
        const int bk = ((lane >> 3) & 1) * 8;
        if (resident && !ptx::mbar_wait(wbar, 0)) timed_out = true;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const Tile tl = get_tile(tile);
            if (tl.rows == 0) continue;
            const bool active = m0 < tl.rows;

            // epilogue operands, fetched now so that their latency hides behind the K loop
            const int my_row = m0 + (lane & 15);
            const int64_t my_tok =
                (ni == 0 && active && my_row < tl.rows) ? (perm ? perm[tl.start + my_row] : tl.start + my_row) : -1;
            float2 bias2[NP / 8];
#pragma unroll
            for (int nt = 0; nt < NP / 8; ++nt)
                bias2[nt] = ni == 0 ? __ldg(reinterpret_cast<const float2*>(bimg + (int64_t)tl.bin * NP + nt * 8 + 2 * q4))
                                    : make_float2(0.0f, 0.0f);

            float acc[NP / 8][4];
#pragma unroll
            for (int nt = 0; nt < NP / 8; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[nt][c] = 0.0f;

            for (int u = 0; u < U1; ++u) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                if (active) {
                    const uint32_t xs = ptx::smem_addr(stages + stage * stage_stride);
                    const uint32_t ws = resident ? ptx::smem_addr(wres + u * L::kWStageBytes) : xs + kTM * kXRowBytes;
                    const uint32_t a_base = xs + (m0 + (lane & 15)) * kXRowBytes + (lane >> 4) * 16;
#pragma unroll
                    for (int kq = 0; kq < (kKS / 16) / kDescentKSplit; ++kq) {
                        const int ks = kq * kDescentKSplit + ni;
                        uint32_t a0, a1, a2, a3;
                        ptx::ldmatrix_x4(a_base + ks * 32, a0, a1, a2, a3);
                        const int kcol = ks * 16 + bk;
                        const int sb = kcol >> 6, kc = kcol & 63;
#pragma unroll
                        for (int np = 0; np < NP / 16; ++np) {
                            const int n = np * 16 + bn;
                            uint32_t b0, b1, b2, b3;
                            ptx::ldmatrix_x4(ws + ptx::swz128((uint32_t)((sb * NP + n) * 128 + kc * 2)), b0, b1, b2, b3);
                            ptx::mma_bf16(acc[2 * np], a0, a1, a2, a3, b0, b1);
                            ptx::mma_bf16(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(empty + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }

            // the second warp of the pair hands over its partial sums; the first adds them, lays the 16
            // logit rows out in shared memory, and one lane per row walks the subtree
            if (ni == 1) {
#pragma unroll
                for (int nt = 0; nt < NP / 8; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) pair[(nt * 4 + c) * 32 + lane] = acc[nt][c];
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + mi), "r"(kDescentKSplit * 32) : "memory");
            if (ni == 0) {
#pragma unroll
                for (int nt = 0; nt < NP / 8; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[nt][c] += pair[(nt * 4 + c) * 32 + lane];
                __syncwarp();       // every lane has read its partials before the area is reused for the rows
                if (active) {
#pragma unroll
                    for (int nt = 0; nt < NP / 8; ++nt) {
                        pair[g * L::kLogitRow + nt * 8 + 2 * q4] = acc[nt][0] + bias2[nt].x;
                        pair[g * L::kLogitRow + nt * 8 + 2 * q4 + 1] = acc[nt][1] + bias2[nt].y;
                        pair[(g + 8) * L::kLogitRow + nt * 8 + 2 * q4] = acc[nt][2] + bias2[nt].x;
                        pair[(g + 8) * L::kLogitRow + nt * 8 + 2 * q4 + 1] = acc[nt][3] + bias2[nt].y;
                    }
                    __syncwarp();
                    if (lane < 16 && my_tok >= 0) {
                        const float* row = pair + lane * L::kLogitRow;
                        int p = 0;
                        for (int r = 0; r < k; ++r) p = 2 * p + 1 + (row[p] >= 0.0f ? 1 : 0);
                        pos_out[my_tok] = (tl.bin << k) + (p - ((1 << k) - 1));
                    }
                    __syncwarp();
                }
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + mi), "r"(kDescentKSplit * 32) : "memory");
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let bulk copies still in flight land before exit
    }
}

}  // namespace fff
