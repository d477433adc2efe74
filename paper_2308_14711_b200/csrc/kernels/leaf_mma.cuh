// Grouped leaf evaluation on tensor cores (bf16, float32 accumulate) with un-permuting write-back.
//
// Algorithm 1, FORWARD_I, leaf branch, for the tokens of one bucket at a time:
//     H = act(X[T_j] W1_j^T + b1_j)        [|T_j|, l]     (GEMM1, K = D)
//     Y = H W2_j^T + b2_j                  [|T_j|, O]     (GEMM2, K = l)
// and row i of Y is stored at the original position of token T_j[i].
//
// Work unit: a tile = up to TM consecutive entries of one bucket.  CTAs are persistent and walk the
// device-built tile list with a static stride.  Inside a CTA the producer warps stream operands into a
// ring of shared-memory stages (cp.async for the gathered token rows, 1-D bulk (TMA) copies for the
// weight images) whose stages complete on mbarriers; 8 consumer warps run both GEMMs with
// mma.sync.m16n8k16, keeping H in registers between them (the accumulator fragment of GEMM1 is the A
// fragment of GEMM2).
//
// Ring contents, in order, per tile:
//   D/kKS   GEMM1 stages: kKS columns of the gathered token rows (16-byte cp.async, rows padded by
//           16 bytes in shared memory so that ldmatrix is conflict-free) + the matching slice of W1_j
//           (one bulk copy of a pre-swizzled image);
//   O/kNC   GEMM2 stages: kNC rows of W2_j (pre-swizzled image) followed by their float32 biases.
// The images are written once at handle creation (repack kernels below).
//
// Requirements: bf16, D % kKS == 0, O % 8 == 0, l <= 64 (padded to kLP in {16, 32, 64} with zero
// weights: act(0) * 0 contributes nothing).
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kKS = 128;         // K columns per GEMM1 stage
constexpr int kNC = 256;         // output columns per GEMM2 stage
// A warp needs about 70 cycles per bulk-copy request whatever its size, which is far too slow for
// one 256-byte request per gathered row.  The token rows are therefore copied with 16-byte cp.async
// by all threads of the producer warps (16 threads per row piece); bulk copies are kept for the
// weight images, where one request moves kilobytes.
constexpr int kProducerWarps = 2;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kRowsPerPass = kProducerThreads / 16;       // rows covered by one cp.async of every producer thread
constexpr int kXRowBytes = kKS * 2 + 16;                    // padded row of a GEMM1 stage
constexpr int kMaxStages = 8;

// A single warp issues dependent instructions only every few cycles, so the arithmetic of a tile is
// spread over 8 consumer warps whatever the tile height: warp (mi, ni) owns the 16 rows of m-tile mi
// and takes every kNSplit-th k-step of GEMM1 (partial sums are added up through shared memory) and
// the ni-th slice of the output columns of every GEMM2 stage.
constexpr int kLeafConsumers = 8;
constexpr int kOutBlock = 64;                               // outputs accumulated at once per warp
constexpr int kOutRowBytes = kOutBlock * 2 + 16;            // padded row of the store staging buffer

// LP: padded hidden width.  TM: token rows per tile (32 or 64).  S: ring stages.
template <int LP, int TM, int S> struct LeafMmaLayout {
    static constexpr int kMTiles = TM / 16;
    static constexpr int kNSplit = kLeafConsumers / kMTiles;
    static constexpr int kThreads = (kLeafConsumers + kProducerWarps) * 32;
    static constexpr int kW1StageBytes = LP * kKS * 2;
    static constexpr int kStage1Bytes = TM * kXRowBytes + kW1StageBytes;
    static constexpr int kW2Bytes = kNC * LP * 2;
    static constexpr int kStage2Bytes = kW2Bytes + kNC * 4;             // weights + float32 biases
    static constexpr int kStageBytes = kStage1Bytes > kStage2Bytes ? kStage1Bytes : kStage2Bytes;
    static constexpr int kStageStride = (kStageBytes + 127) & ~127;
    // per consumer warp: y staging (16 padded rows), also used to exchange the GEMM1 partial sums
    static constexpr int kWarpScratch = (16 * kOutRowBytes > LP * 64 ? 16 * kOutRowBytes : LP * 64);
    static constexpr int kStagingBytes = kLeafConsumers * kWarpScratch;
    static constexpr int kSmemBytes = S * kStageStride + kStagingBytes + 128 /* barriers */ + 128 /* align */;
    static_assert(S <= kMaxStages, "barrier area holds 2 * kMaxStages mbarriers");
    static_assert((kKS / 16) % kNSplit == 0 && (kNC / kOutBlock) % kNSplit == 0, "split must divide the stage");
};

// ---- one-time repacking of the leaf parameters into stage images --------------------------------

// W1 image: [leaf][D/kKS stages][kKS/64 sub-blocks][LP rows][64 columns], 128-byte swizzled.
template <typename T>
__global__ void k_pack_w1(const T* __restrict__ w1, __nv_bfloat16* __restrict__ img, int n_leaves, int l, int LP, int D)
{
    const int64_t total = (int64_t)n_leaves * LP * D;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int k = (int)(i % D);
        const int n = (int)((i / D) % LP);
        const int64_t j = i / ((int64_t)D * LP);
        const int u = k / kKS, sb = (k % kKS) / 64, kc = k % 64;
        const uint32_t off = ptx::swz128((uint32_t)((sb * LP + n) * 128 + kc * 2));
        const int64_t base = (j * (D / kKS) + u) * (int64_t)(LP * kKS);          // elements
        const float v = n < l ? Elem<T>::to_float(w1[(j * l + n) * (int64_t)D + k]) : 0.0f;
        img[base + off / 2] = __float2bfloat16_rn(v);
    }
}

// W2 image: [leaf][ceil(O/kNC) stages]{ [kNC rows][LP columns] 128-byte swizzled, then kNC float32 biases }.
template <typename T>
__global__ void k_pack_w2(const T* __restrict__ w2, const T* __restrict__ b2, unsigned char* __restrict__ img,
                          int n_leaves, int l, int LP, int O)
{
    const int U2 = (O + kNC - 1) / kNC;
    const int64_t stage_bytes = (int64_t)kNC * LP * 2 + kNC * 4;
    const int64_t total = (int64_t)n_leaves * U2 * kNC * (LP + 1);       // LP weights + 1 bias per row
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % (LP + 1));
        const int n = (int)((i / (LP + 1)) % kNC);
        const int64_t ju = i / ((int64_t)(LP + 1) * kNC);                  // leaf * U2 + stage
        const int64_t j = ju / U2;
        const int o = (int)(ju % U2) * kNC + n;
        unsigned char* st = img + ju * stage_bytes;
        if (c < LP) {
            const float v = (o < O && c < l) ? Elem<T>::to_float(w2[(j * O + o) * (int64_t)l + c]) : 0.0f;
            const uint32_t off = ptx::swz128((uint32_t)(n * LP * 2 + c * 2));
            *reinterpret_cast<__nv_bfloat16*>(st + off) = __float2bfloat16_rn(v);
        } else {
            reinterpret_cast<float*>(st + (int64_t)kNC * LP * 2)[n] = o < O ? Elem<T>::to_float(b2[j * O + o]) : 0.0f;
        }
    }
}

// b1 image: [leaf][LP] float32, zero beyond l.
template <typename T>
__global__ void k_pack_b1(const T* __restrict__ b1, float* __restrict__ img, int n_leaves, int l, int LP)
{
    const int64_t total = (int64_t)n_leaves * LP;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % LP);
        const int64_t j = i / LP;
        img[i] = n < l ? Elem<T>::to_float(b1[j * l + n]) : 0.0f;
    }
}

// ---- the kernel ------------------------------------------------------------------------------------

template <int LP, int TM, int S>
__global__ void __launch_bounds__((kLeafConsumers + kProducerWarps) * 32, LP <= 32 ? 2 : 1)
k_leaf_mma(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ perm,
           const Tile* __restrict__ tiles, int n_tiles_total,
           const __nv_bfloat16* __restrict__ w1img, const float* __restrict__ b1img,
           const unsigned char* __restrict__ w2img, __nv_bfloat16* __restrict__ y,
           int D, int O, int act, int* __restrict__ status)
{
    using L = LeafMmaLayout<LP, TM, S>;
    constexpr int kStages = S;
    constexpr int kTM = TM;
    constexpr int kMTiles = L::kMTiles;
    constexpr int kNSplit = L::kNSplit;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    unsigned char* stages = smem;
    unsigned char* staging = smem + kStages * L::kStageStride;
    uint64_t* full = reinterpret_cast<uint64_t*>(staging + L::kStagingBytes);
    uint64_t* empty = full + kStages;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int U1 = D / kKS;
    const int U2 = (O + kNC - 1) / kNC;
    const int ntiles = n_tiles_total;      // the list may contain empty tiles (rows = 0)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, kProducerThreads + 1);     // every producer thread + the weight copy
            ptx::mbar_init(empty + s, kLeafConsumers);
        }
        ptx::fence_mbar_init();
    }
    pdl_trigger();
    __syncthreads();
    pdl_wait();

    int stage = 0;
    uint32_t phase = 0;
    bool timed_out = false;

    if (warp >= kLeafConsumers) {
        // ------------------------------------------------------------------ producer warps
        const int ptid = threadIdx.x - kLeafConsumers * 32;
        const int prow = ptid >> 4, pchunk = ptid & 15;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const Tile tl = tiles[tile];
            if (tl.rows == 0) continue;
            const __nv_bfloat16* src[kTM / kRowsPerPass];
#pragma unroll
            for (int i = 0; i < kTM / kRowsPerPass; ++i) {
                const int r = i * kRowsPerPass + prow;
                src[i] = r < tl.rows ? x + (int64_t)perm[tl.start + r] * D + pchunk * 8 : nullptr;
            }
            for (int u = 0; u < U1; ++u) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                unsigned char* st = stages + stage * L::kStageStride;
                if (ptid == 0) {
                    ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)L::kW1StageBytes);
                    ptx::bulk_g2s(st + kTM * kXRowBytes, w1img + ((int64_t)tl.bin * U1 + u) * (LP * kKS), L::kW1StageBytes,
                                  full + stage);
                }
#pragma unroll
                for (int i = 0; i < kTM / kRowsPerPass; ++i)
                    if (src[i]) ptx::cp_async16(st + (i * kRowsPerPass + prow) * kXRowBytes + pchunk * 16, src[i] + u * kKS);
                ptx::cp_async_mbar_arrive(full + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
            for (int u = 0; u < U2; ++u) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                if (ptid == 0) {
                    ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)L::kStage2Bytes);
                    ptx::bulk_g2s(stages + stage * L::kStageStride, w2img + ((int64_t)tl.bin * U2 + u) * L::kStage2Bytes,
                                  L::kStage2Bytes, full + stage);
                }
                ptx::mbar_arrive(full + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int mi = warp % kMTiles, ni = warp / kMTiles;
        const int m0 = mi * 16;
        unsigned char* my_scratch = staging + warp * L::kWarpScratch;
        const int g = lane >> 2, q4 = lane & 3;
        const int bn = (lane & 7) + ((lane >> 4) << 3);
        const int bk = ((lane >> 3) & 1) * 8;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const Tile tl = tiles[tile];
            if (tl.rows == 0) continue;
            const bool active = m0 < tl.rows;          // m-tiles without valid rows only keep the ring moving

            // epilogue operands, fetched now so that their latency hides behind the K loop
            const int my_row = m0 + (lane & 15);
            const int64_t my_tok = (active && my_row < tl.rows) ? perm[tl.start + my_row] : -1;
            float2 b1r[LP / 8];
#pragma unroll
            for (int nt = 0; nt < LP / 8; ++nt)
                b1r[nt] = __ldg(reinterpret_cast<const float2*>(b1img + (int64_t)tl.bin * LP + nt * 8 + 2 * q4));

            // GEMM1, this warp's share of the k-steps: acc1[nt] += X[m0..m0+16) . W1[nt*8 .. nt*8+8)^T
            float acc1[LP / 8][4];
#pragma unroll
            for (int nt = 0; nt < LP / 8; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc1[nt][c] = 0.0f;

            for (int u = 0; u < U1; ++u) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                if (active) {
                    const uint32_t xs = ptx::smem_addr(stages + stage * L::kStageStride);
                    const uint32_t ws = xs + kTM * kXRowBytes;
                    const uint32_t a_base = xs + (m0 + (lane & 15)) * kXRowBytes + (lane >> 4) * 16;
#pragma unroll
                    for (int kq = 0; kq < (kKS / 16) / kNSplit; ++kq) {
                        const int ks = kq * kNSplit + ni;
                        uint32_t a0, a1, a2, a3;
                        ptx::ldmatrix_x4(a_base + ks * 32, a0, a1, a2, a3);
                        const int kcol = ks * 16 + bk;
                        const int sb = kcol >> 6, kc = kcol & 63;
#pragma unroll
                        for (int np = 0; np < LP / 16; ++np) {
                            const int n = np * 16 + bn;
                            uint32_t b0, b1, b2, b3;
                            ptx::ldmatrix_x4(ws + ptx::swz128((uint32_t)((sb * LP + n) * 128 + kc * 2)), b0, b1, b2, b3);
                            ptx::mma_bf16(acc1[2 * np], a0, a1, a2, a3, b0, b1);
                            ptx::mma_bf16(acc1[2 * np + 1], a0, a1, a2, a3, b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(empty + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }

            // add up the partial sums of the kNSplit warps that share this m-tile (through shared memory),
            // then bias + activation; H stays in registers as the A operand of GEMM2
            {
                float* mine = reinterpret_cast<float*>(my_scratch);
#pragma unroll
                for (int nt = 0; nt < LP / 8; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) mine[(nt * 4 + c) * 32 + lane] = acc1[nt][c];
                asm volatile("bar.sync %0, %1;" ::"r"(1 + mi), "r"(kNSplit * 32) : "memory");
#pragma unroll
                for (int j = 1; j < kNSplit; ++j) {
                    const float* other =
                        reinterpret_cast<const float*>(staging + (mi + kMTiles * ((ni + j) % kNSplit)) * L::kWarpScratch);
#pragma unroll
                    for (int nt = 0; nt < LP / 8; ++nt)
#pragma unroll
                        for (int c = 0; c < 4; ++c) acc1[nt][c] += other[(nt * 4 + c) * 32 + lane];
                }
                asm volatile("bar.sync %0, %1;" ::"r"(1 + mi), "r"(kNSplit * 32) : "memory");
            }
            uint32_t hA[LP / 8][2];
#pragma unroll
            for (int nt = 0; nt < LP / 8; ++nt) {
                const float2 b = b1r[nt];
                hA[nt][0] = ptx::pack_bf16(activate(act, acc1[nt][0] + b.x), activate(act, acc1[nt][1] + b.y));
                hA[nt][1] = ptx::pack_bf16(activate(act, acc1[nt][2] + b.x), activate(act, acc1[nt][3] + b.y));
            }

            // GEMM2 + bias + store, this warp's slice of the output columns of every stage
            for (int u = 0; u < U2; ++u) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                if (active) {
                    const unsigned char* st = stages + stage * L::kStageStride;
                    const uint32_t ws = ptx::smem_addr(st);
                    const float* bias = reinterpret_cast<const float*>(st + L::kW2Bytes);
#pragma unroll 1
                    for (int blk = 0; blk < (kNC / kOutBlock) / kNSplit; ++blk) {
                        const int c0 = (ni * ((kNC / kOutBlock) / kNSplit) + blk) * kOutBlock;    // first column inside the stage
                        const int o_base = u * kNC + c0;
                        if (o_base >= O) break;
                        float acc2[kOutBlock / 8][4];
#pragma unroll
                        for (int nt = 0; nt < kOutBlock / 8; ++nt)
#pragma unroll
                            for (int c = 0; c < 4; ++c) acc2[nt][c] = 0.0f;
#pragma unroll
                        for (int np = 0; np < kOutBlock / 16; ++np) {
                            const int n = c0 + np * 16 + bn;
#pragma unroll
                            for (int kk = 0; kk < LP / 16; ++kk) {
                                uint32_t b0, b1, b2, b3;
                                ptx::ldmatrix_x4(ws + ptx::swz128((uint32_t)(n * LP * 2 + (kk * 16 + bk) * 2)), b0, b1, b2, b3);
                                ptx::mma_bf16(acc2[2 * np], hA[2 * kk][0], hA[2 * kk][1], hA[2 * kk + 1][0], hA[2 * kk + 1][1], b0, b1);
                                ptx::mma_bf16(acc2[2 * np + 1], hA[2 * kk][0], hA[2 * kk][1], hA[2 * kk + 1][0], hA[2 * kk + 1][1], b2, b3);
                            }
                        }
                        // fragments -> padded staging rows (bf16), then whole 16-byte units to y
#pragma unroll
                        for (int nt = 0; nt < kOutBlock / 8; ++nt) {
                            const float2 b = *reinterpret_cast<const float2*>(bias + c0 + nt * 8 + 2 * q4);
                            *reinterpret_cast<uint32_t*>(my_scratch + g * kOutRowBytes + nt * 16 + q4 * 4) =
                                ptx::pack_bf16(acc2[nt][0] + b.x, acc2[nt][1] + b.y);
                            *reinterpret_cast<uint32_t*>(my_scratch + (g + 8) * kOutRowBytes + nt * 16 + q4 * 4) =
                                ptx::pack_bf16(acc2[nt][2] + b.x, acc2[nt][3] + b.y);
                        }
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const int r = it * 4 + (lane >> 3);
                            const int unit = lane & 7;
                            const int o = o_base + unit * 8;
                            const int64_t t = __shfl_sync(kFullMask, my_tok, r);
                            if (t >= 0 && o < O) {
                                const uint4 v = *reinterpret_cast<const uint4*>(my_scratch + r * kOutRowBytes + unit * 16);
                                __stcs(reinterpret_cast<uint4*>(y + t * O + o), v);
                            }
                        }
                        __syncwarp();
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(empty + stage);
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let bulk copies still in flight land before exit
    }
}

}  // namespace fff
