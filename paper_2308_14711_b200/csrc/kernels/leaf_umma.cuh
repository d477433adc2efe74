// Grouped leaf evaluation on the fifth-generation tensor cores (tcgen05, bf16 -> float32) with
// un-permuting write-back.
//
// Algorithm 1, FORWARD_I, leaf branch, for the tokens of one bucket at a time:
//     H = act(X[T_j] W1_j^T + b1_j)        [|T_j|, l]     (GEMM1, K = D)
//     Y = H W2_j^T + b2_j                  [|T_j|, O]     (GEMM2, K = l)
// and row i of Y is stored at the original position of token T_j[i].
//
// Work unit: a tile = up to 128 consecutive entries of one bucket = the 128 rows of one tcgen05.mma.
// One persistent CTA per SM takes tiles from a device-wide counter, in list order.  Warp roles:
//   warps 0-7   epilogue.  A thread owns one token row (= one tensor-memory lane; warps w and w + 4
//               share the lanes of quarter w % 4) and one half of the columns: H = act(acc1 + b1) to
//               shared memory as the A operand of GEMM2; then, per piece of 128 output columns,
//               acc2 + b2 -> bf16 -> 32-byte stores straight to the token's row of y.  Two warps per
//               quarter measured faster than one, three (with 96-column pieces) and four; quarters
//               without valid rows (short tiles) only keep the barriers moving;
//   warp 8      tile scheduler: claims list entries with an atomic counter, skips empty ones and
//               publishes them through a small shared-memory queue.  A tile is claimed only when the
//               gathers have started on the one before it: claiming further ahead would hand a CTA
//               work long before it can do it and leave other SMs idle at the end;
//   warp 9      GEMM1 issuer: per K-block of 64 columns four tcgen05.mma (M = 128, N = LP, K = 16);
//   warp 10     GEMM2: bulk copies of the W2 pieces (each followed by its 128 float32 biases) into
//               their own ring and, per piece, LP/16 tcgen05.mma (M = 128, N = 128) into one of two
//               accumulators;
//   warps 11-14 gather of the token rows: per K-block one tile::gather4 tensor-map load per 4 rows
//               (4 x 128 bytes, 128-byte swizzled by the copy engine), the 4-row groups dealt
//               round-robin to the four warps; the first of them also starts the bulk copy of the
//               matching W1 K-block.
// GEMM1 of the next tile runs while the epilogue of the current one drains, and the row gathers never
// stop in between: loads and stores overlap across tiles.
//
// When the hidden width is padded (l < LP) the spare column l of H is set to 1 and the same column of the W2
// image holds b2, so GEMM2 adds the output bias itself and the epilogue only converts and stores; with
// l == LP the biases ride behind the W2 pieces and are added in the epilogue.
//
// Rows of a ragged tile beyond its length are not loaded: their accumulator rows hold garbage that is
// never stored (rows of an MMA are independent).
// Tiles of at most 64 (32) rows are stacked twice (four times) in the MMA rows of GEMM2 so that every epilogue
// warp has a share of their columns (see the epilogue).
//
// Every wait is bounded (see ptx.cuh); tensor memory is released on every exit path.
//
// Requirements: bf16, D % 128 == 0, O % 16 == 0, l <= 64 (padded to LP in {16, 32, 64}), x 16-byte aligned.
#pragma once

#include <cuda.h>      // CUtensorMap

#include "common.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kLUM = 128;                  // token rows per tile
constexpr int kLUKB = 64;                  // columns per K-block of GEMM1
constexpr int kLUPiece = 128;              // output columns per GEMM2 piece
constexpr int kLUAccStride = 128;          // tensor-memory columns between the two GEMM2 accumulators
constexpr int kLUEpiWarps = 8;
constexpr int kLUColParts = kLUEpiWarps / 4;       // epilogue warps per lane quarter = column parts per piece
constexpr int kLUHParts = 2;                       // of which this many compute H
static_assert(kLUPiece % (32 * kLUColParts) == 0, "whole 32-column tensor-memory loads per piece and thread");
constexpr int kLUGatherWarps = 4;
constexpr int kLUSchedWarp = kLUEpiWarps, kLUGemm1Warp = kLUEpiWarps + 1, kLUGemm2Warp = kLUEpiWarps + 2;
constexpr int kLUFirstGatherWarp = kLUEpiWarps + 3;
constexpr int kLUWarps = kLUEpiWarps + 3 + kLUGatherWarps;
constexpr int kLUThreads = kLUWarps * 32;
constexpr int kLUMaxStages = 8;
constexpr int kLUMaxW2Slots = 12;
constexpr int kLUQueue = 4;                // tiles published ahead by the scheduler
constexpr int kLUConsumerWarps = kLUWarps - 1;     // every warp but the scheduler reads the tile queue
constexpr int kLUTmemCols = 512;

// kW8: the leaf weights are stored as 8-bit floats (e4m3 codes, one float32 scale per leaf and matrix).  The MMA wants
// both operands as bf16, so the codes land in a staging part of their ring slot and the warp that issues the MMAs
// expands them (every code is exactly a bf16 value) into the operand layout first; the scales multiply the
// accumulators in the epilogue.
// GL: leaves per tile.  1: a tile holds tokens of one leaf.  8: a tile holds tokens of one node three levels above the
// leaves; GEMM1 then runs against the hidden units of that node's 8 leaves side by side plus the 7 nodes of its
// subtree (N = 8 LP + 16 columns, the last 9 zero), the epilogue walks the three levels from the node logits, keeps
// each row's own leaf's LP columns of H and zeroes the others, and GEMM2 contracts over all 8 LP columns against the
// 8 leaves' output weights.  The tokens' rows then cross the memory system twice in all (first stage of the descent,
// then here) instead of being gathered once more per level group, and tiles are as full as the node's share of the batch.
template <int LP, bool kW8 = false, int GL = 1> struct LeafUmmaLayout {
    static_assert(LP == 16 || LP == 32 || LP == 64, "padded hidden width");
    static_assert(GL == 1 || (GL == 8 && LP == 16 && !kW8), "grouped tiles: 8 leaves of padded width 16, bf16 weights");
    static constexpr int kN1 = GL == 1 ? LP : GL * LP + 16;                  // columns of GEMM1
    static constexpr int kHCols = GL * LP;                                   // K of GEMM2
    static constexpr int kRowBytes = GL == 1 ? LP * 2 : 128;                 // row of H and of a W2 piece (per K-block of 64 columns when grouped)
    static constexpr int kHBlocks = kHCols * 2 / kRowBytes;                  // K-blocks of H and of a W2 piece
    // A ring stage holds kSub K-blocks of 64 columns (each a 128-byte swizzled operand tile of its own):
    // every stage costs each role a fixed few hundred cycles of barrier traffic, so two K-blocks share one
    // where shared memory allows.
    static constexpr int kSub = GL > 1 ? 1 : LP <= 32 ? 2 : 1;
    static constexpr int kXSubBytes = kLUM * kLUKB * 2;
    static constexpr int kW1SubBytes = kN1 * kLUKB * 2;
    static constexpr int kXStageBytes = kSub * kXSubBytes;
    static constexpr int kW1StageBytes = kSub * kW1SubBytes;
    static constexpr int kW1CodeBytes = kW8 ? kW1StageBytes / 2 : 0;         // staging for the codes of the stage's W1 K-blocks
    static constexpr int kW1CopyBytes = kW8 ? kW1CodeBytes : kW1StageBytes;  // what the bulk copy of a stage brings
    static constexpr int kStageBytes = kXStageBytes + kW1StageBytes + kW1CodeBytes;      // a multiple of 1024
    static constexpr int kW2Bytes = kLUPiece * kHCols * 2;                   // weights of a piece (bf16 operand)
    static constexpr int kW2CodeBytes = kW8 ? kW2Bytes / 2 : 0;
    static constexpr int kW2BiasOff = kW2Bytes + kW2CodeBytes;               // the piece's 128 float32 biases inside a slot
    static constexpr int kW2CopyOff = kW8 ? kW2Bytes : 0;                    // where the bulk copy of a piece lands in its slot
    static constexpr int kW2PieceBytes = (kW8 ? kW2CodeBytes : kW2Bytes) + kLUPiece * 4;    // a piece in the image: weights + biases
    static constexpr int kW2SlotStride = (kW2BiasOff + kLUPiece * 4 + 1023) & ~1023;
    static constexpr int kHBytes = kLUM * kHCols * 2;
    // W2 ring: a whole tile's pieces (O <= 1024) when they are small, so that no copy waits for an MMA just issued
    static constexpr int kW2Slots = GL > 1 ? 3 : LP <= 16 ? 8 : LP <= 32 ? (kW8 ? 6 : 8) : 4;
    static constexpr int kAcc2Col = GL > 1 ? 256 : 64;                       // first tensor-memory column of the two GEMM2 accumulators
    static constexpr int kBarrierBytes = 640;
    static constexpr int smem_bytes(int stages) {
        return 1024 + stages * kStageBytes + kW2Slots * kW2SlotStride + kHBytes + kBarrierBytes;
    }
};

// Swizzle of a byte offset inside an operand tile whose rows are row_bytes (32, 64 or 128) long: the
// 16-byte unit index inside a row is XORed with bits of the 128-byte line index, as the 32-, 64- and
// 128-byte swizzle modes of the tensor cores expect.
__host__ __device__ __forceinline__ uint32_t swz_rows(uint32_t off, int row_bytes) {
    return off ^ (((off >> 7) & (uint32_t)(row_bytes / 16 - 1)) << 4);
}

// W2 image for GEMM2: [leaf][ceil(O/128) pieces]{ [128 rows (output features)][LP columns] swizzled,
// then the 128 float32 biases of those features }.
template <typename T>
__global__ void k_pack_w2_umma(const T* __restrict__ w2, const T* __restrict__ b2, unsigned char* __restrict__ img,
                               int n_leaves, int l, int LP, int O)
{
    const int P = (O + kLUPiece - 1) / kLUPiece;
    const int64_t piece_bytes = (int64_t)kLUPiece * LP * 2 + kLUPiece * 4;
    const int64_t total = (int64_t)n_leaves * P * kLUPiece * (LP + 1);      // LP weights + 1 bias per row
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % (LP + 1));
        const int n = (int)((i / (LP + 1)) % kLUPiece);
        const int64_t jp = i / ((int64_t)(LP + 1) * kLUPiece);             // leaf * P + piece
        const int64_t j = jp / P;
        const int o = (int)(jp % P) * kLUPiece + n;
        unsigned char* piece = img + jp * piece_bytes;
        if (c < LP) {
            // a spare padded column (l < LP) carries the output bias: H gets a constant 1 there, so GEMM2 adds
            // b2 by itself and the epilogue has no bias to fetch and add (b2 is bf16 already: exact)
            float v = (o < O && c < l) ? Elem<T>::to_float(w2[(j * O + o) * (int64_t)l + c]) : 0.0f;
            if (c == l && o < O) v = Elem<T>::to_float(b2[j * O + o]);
            *reinterpret_cast<__nv_bfloat16*>(piece + swz_rows((uint32_t)(n * LP * 2 + c * 2), LP * 2)) = __float2bfloat16_rn(v);
        } else {
            const float v = o < O ? Elem<T>::to_float(b2[j * O + o]) : 0.0f;
            reinterpret_cast<float*>(piece + (int64_t)kLUPiece * LP * 2)[n] = v;
        }
    }
}

// Images for grouped tiles (kLUGroup = 8 leaves per tile): bin g is node g of level depth - 3, N1 = 8 LP + 16.
//   w1g  [bin][D / 64][N1 rows][64 columns] 128-byte swizzled: row j LP + u = hidden unit u of leaf 8 g + j (zero for
//        u >= l); rows 8 LP + q, q < 7: node q of the subtree below node g, breadth-first; the other rows zero;
//   g1b  [bin][N1] float32: the biases of those rows;
//   w2g  [bin][ceil(O / 128) pieces]{ 2 K-blocks of [128 rows (output features)][64 columns] 128-byte swizzled, then 128
//        float32 (unused, zero) }: column j LP + u of feature o is w2[8 g + j][o][u], and for u == l (the spare hidden
//        column, which H sets to 1) the output bias b2[8 g + j][o].  The image is zeroed before this kernel runs.
constexpr int kLUGroup = 8;
template <typename T>
__global__ void k_pack_leaf_groups(const T* __restrict__ w1, const T* __restrict__ b1, const T* __restrict__ w2, const T* __restrict__ b2,
                                   const T* __restrict__ node_w, const T* __restrict__ node_b, __nv_bfloat16* __restrict__ w1g,
                                   float* __restrict__ g1b, unsigned char* __restrict__ w2g, int n_bins, int depth, int l, int LP, int D,
                                   int O)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int HC = kLUGroup * LP, N1 = HC + 16;
    // node q of the subtree below (level depth - 3, position g), as an index into node_w / node_b
    auto node_of = [&](int64_t g, int q) {
        const int r = q == 0 ? 0 : q < 3 ? 1 : 2;
        return (((int64_t)1 << (depth - 3 + r)) - 1) + (g << r) + (q - ((1 << r) - 1));
    };
    for (int64_t i = t0; i < (int64_t)n_bins * N1 * D; i += stride) {
        const int k = (int)(i % D), n = (int)((i / D) % N1);
        const int64_t g = i / ((int64_t)D * N1);
        float v = 0.0f;
        if (n < HC) {
            const int j = n / LP, u = n % LP;
            if (u < l) v = Elem<T>::to_float(w1[((g * kLUGroup + j) * l + u) * (int64_t)D + k]);
        } else if (n - HC < 7) {
            v = Elem<T>::to_float(node_w[node_of(g, n - HC) * D + k]);
        }
        const int64_t base = (g * (D / kLUKB) + k / kLUKB) * (int64_t)(N1 * kLUKB);       // elements
        w1g[base + ptx::swz128((uint32_t)(n * 128 + (k % kLUKB) * 2)) / 2] = __float2bfloat16_rn(v);
    }
    for (int64_t i = t0; i < (int64_t)n_bins * N1; i += stride) {
        const int n = (int)(i % N1);
        const int64_t g = i / N1;
        float v = 0.0f;
        if (n < HC) {
            const int j = n / LP, u = n % LP;
            if (u < l && b1) v = Elem<T>::to_float(b1[(g * kLUGroup + j) * l + u]);
        } else if (n - HC < 7 && node_b) {
            v = Elem<T>::to_float(node_b[node_of(g, n - HC)]);
        }
        g1b[i] = v;
    }
    const int P = (O + kLUPiece - 1) / kLUPiece;
    const int64_t piece_bytes = (int64_t)kLUPiece * HC * 2 + kLUPiece * 4;
    for (int64_t i = t0; i < (int64_t)n_bins * P * kLUPiece * HC; i += stride) {
        const int c = (int)(i % HC), n = (int)((i / HC) % kLUPiece);
        const int64_t gp = i / ((int64_t)HC * kLUPiece), g = gp / P;
        const int o = (int)(gp % P) * kLUPiece + n, j = c / LP, u = c % LP;
        float v = 0.0f;
        if (o < O) {
            if (u < l) v = Elem<T>::to_float(w2[((g * kLUGroup + j) * O + o) * (int64_t)l + u]);
            else if (u == l && b2) v = Elem<T>::to_float(b2[(g * kLUGroup + j) * O + o]);
        }
        unsigned char* blk = w2g + gp * piece_bytes + (int64_t)(c / kLUKB) * (kLUPiece * 128);
        *reinterpret_cast<__nv_bfloat16*>(blk + ptx::swz128((uint32_t)(n * 128 + (c % kLUKB) * 2))) = __float2bfloat16_rn(v);
    }
}

// Images of 8-bit leaf weights: w1c [leaf][D / 64][LP][64] codes (rows past l zero = the code of +0);
// w2c [leaf][ceil(O/128) pieces]{ [128 rows (output features)][LP] codes, then their 128 float32 biases }.
template <typename T>
__global__ void k_pack_leaf_codes(const unsigned char* __restrict__ w1, const unsigned char* __restrict__ w2, const T* __restrict__ b2,
                                  unsigned char* __restrict__ w1c, unsigned char* __restrict__ w2c, int n_leaves, int l, int LP,
                                  int D, int O)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int KBn = D / kLUKB;
    for (int64_t i = t0; i < (int64_t)n_leaves * KBn * LP * kLUKB; i += stride) {
        const int c = (int)(i % kLUKB), r = (int)((i / kLUKB) % LP);
        const int64_t kb = (i / ((int64_t)kLUKB * LP)) % KBn, j = i / ((int64_t)kLUKB * LP * KBn);
        w1c[i] = r < l ? w1[(j * l + r) * D + kb * kLUKB + c] : (unsigned char)0;
    }
    const int P = (O + kLUPiece - 1) / kLUPiece;
    const int64_t piece_bytes = (int64_t)kLUPiece * LP + kLUPiece * 4;
    for (int64_t i = t0; i < (int64_t)n_leaves * P * kLUPiece * (LP + 1); i += stride) {
        const int c = (int)(i % (LP + 1)), n = (int)((i / (LP + 1)) % kLUPiece);
        const int64_t jp = i / ((int64_t)(LP + 1) * kLUPiece), j = jp / P;
        const int o = (int)(jp % P) * kLUPiece + n;
        unsigned char* piece = w2c + jp * piece_bytes;
        if (c < LP) piece[n * LP + c] = (o < O && c < l) ? w2[(j * O + o) * (int64_t)l + c] : (unsigned char)0;
        else reinterpret_cast<float*>(piece + (int64_t)kLUPiece * LP)[n] = (o < O && b2) ? Elem<T>::to_float(b2[j * O + o]) : 0.0f;
    }
}

// Two e4m3 codes (the low and the high byte of `pair`) as two bf16 values: every e4m3 value is exactly a half and
// exactly a bf16 value, so the published conversions e4m3x2 -> f16x2, f16 -> f32, f32x2 -> bf16x2 lose nothing.
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t pair) {
    uint32_t h2, out;
    asm("{\n\t.reg .b16 p;\n\tcvt.u16.u32 p, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, p;\n\t}" : "=r"(h2) : "r"(pair));
    float lo, hi;
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}" : "=f"(lo), "=f"(hi) : "r"(h2));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out) : "f"(hi), "f"(lo));
    return out;
}

// A tile of e4m3 codes, [rows][COLS] row-major, expanded by one warp into the K-major bf16 operand layout with rows of
// 2 COLS bytes, swizzled in the mode of that width.  Units of 16 codes (16 bytes in, two 16-byte units out).
template <int COLS>
__device__ __forceinline__ void expand_e4m3_tile(const unsigned char* __restrict__ src, unsigned char* __restrict__ dst, int rows,
                                                 int lane)
{
    const int n_units = rows * COLS / 16;
#pragma unroll 4
    for (int u = lane; u < n_units; u += 32) {
        const uint4 raw = *reinterpret_cast<const uint4*>(src + u * 16);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o[2 * i] = e4m3x2_to_bf16x2(w[i] & 0xffffu);
            o[2 * i + 1] = e4m3x2_to_bf16x2(w[i] >> 16);
        }
        const uint32_t off = (uint32_t)(u * 16 / COLS) * (COLS * 2) + (uint32_t)(u * 16 % COLS) * 2;
        *reinterpret_cast<uint4*>(dst + swz_rows(off, COLS * 2)) = make_uint4(o[0], o[1], o[2], o[3]);
        *reinterpret_cast<uint4*>(dst + swz_rows(off + 16, COLS * 2)) = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// sched: two ints, both zero before the first launch and again after every launch: [0] list entries
// handed out so far, [1] CTAs that have finished.
// kFold: l < LP, the spare hidden column l carries the output bias (see k_pack_w2_umma).
// slot_counts (optional): instead of a tile list, the lists the descent kernel filled directly (slot_tokens):
// perm[bin * cap + i], i < slot_counts[bin], are the tokens of bin.  The scheduler then derives the tiles itself:
// every lane owns a run of bins and knows how many tiles precede it; a claimed number is resolved by the lane
// whose range holds it.  The last CTA to finish clears the counts for the next call.
// kW8: w1codes / w2img hold e4m3 codes ([leaf][D / 64][LP][64], and per piece [128][LP] codes + 128 float32 biases),
// scale1 / scale2 [leaf] the float32 scales of W1 and W2 (kFold must be off: the biases are added in the epilogue).
// GL = 8 (grouped tiles, see LeafUmmaLayout): a bin is a node three levels above the leaves; w1img holds per bin and
// K-block the 8 LP + 16 rows (hidden units of the 8 leaves, the 7 nodes of the subtree breadth-first, zeros), g1bias
// [bin][8 LP + 16] the matching biases, w2img per bin and piece the 128 x 8 LP output weights in two K-blocks (kFold:
// every leaf's spare column carries its output bias); leaf_out / leaf_out2 (optional) receive every token's leaf.
template <int LP, bool kFold, bool kW8 = false, int GL = 1>
__global__ void __launch_bounds__(kLUThreads, 1)
k_leaf_umma(const __grid_constant__ CUtensorMap tmap_x, const int32_t* __restrict__ perm,
            const Tile* __restrict__ tiles, int n_tiles_total,
            const __nv_bfloat16* __restrict__ w1img, const float* __restrict__ b1img,
            const unsigned char* __restrict__ w2img, __nv_bfloat16* __restrict__ y,
            int D, int O, int l, int act, int kStages, int wide_stores, int passes, int* __restrict__ sched,
            int32_t* __restrict__ slot_counts, int n_bins, int cap, int* __restrict__ status,
            const unsigned char* __restrict__ w1codes, const float* __restrict__ scale1, const float* __restrict__ scale2,
            const float* __restrict__ g1bias, int32_t* __restrict__ leaf_out, int32_t* __restrict__ leaf_out2)
{
    static_assert(!(kW8 && kFold), "8-bit weights take their biases in the epilogue");
    static_assert(GL == 1 || kFold, "grouped tiles take the output bias through the spare hidden column");
    using L = LeafUmmaLayout<LP, kW8, GL>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* w2ring = ring + kStages * L::kStageBytes;
    unsigned char* hbuf = w2ring + L::kW2Slots * L::kW2SlotStride;
    uint64_t* full = reinterpret_cast<uint64_t*>(hbuf + L::kHBytes);
    uint64_t* empty = full + kLUMaxStages;
    uint64_t* w2_full = empty + kLUMaxStages;
    uint64_t* w2_empty = w2_full + kLUMaxW2Slots;
    uint64_t* q_full = w2_empty + kLUMaxW2Slots;
    uint64_t* q_empty = q_full + kLUQueue;
    uint64_t* acc1_full = q_empty + kLUQueue;
    uint64_t* acc1_empty = acc1_full + 1;
    uint64_t* h_full = acc1_empty + 1;
    uint64_t* y_full = h_full + 1;          // [2]
    uint64_t* y_empty = y_full + 2;         // [2]
    Tile* queue = reinterpret_cast<Tile*>(y_empty + 2);                      // [kLUQueue]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(queue + kLUQueue);
    uint64_t* want = reinterpret_cast<uint64_t*>(tmem_slot + 2);             // the gathers have started another tile

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = D / (kLUKB * L::kSub);                   // ring stages per tile
    const int P = (O + kLUPiece - 1) / kLUPiece;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full + s, kLUGatherWarps);           // one arrival per gather warp
            ptx::mbar_init(empty + s, 1);
        }
        for (int s = 0; s < L::kW2Slots; ++s) {
            ptx::mbar_init(w2_full + s, 1);
            ptx::mbar_init(w2_empty + s, 1 + kLUEpiWarps);      // the MMAs that read the weights + every reader of the biases
        }
        for (int s = 0; s < kLUQueue; ++s) {
            ptx::mbar_init(q_full + s, 1);
            ptx::mbar_init(q_empty + s, kLUConsumerWarps);
        }
        ptx::mbar_init(want, 1);
        ptx::mbar_init(acc1_full, 1);
        ptx::mbar_init(acc1_empty, kLUEpiWarps * 32);
        ptx::mbar_init(h_full, kLUEpiWarps * 32);
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(y_full + b, 1);
            ptx::mbar_init(y_empty + b, kLUEpiWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    if (warp == kLUGemm1Warp) {
        ptx::tmem_alloc(tmem_slot, kLUTmemCols);
        ptx::tmem_relinquish_alloc_permit();
    }
    ptx::tc_fence_before_sync();
    pdl_trigger();
    __syncthreads();
    ptx::tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = *tmem_slot;

    bool timed_out = false;
    const int max_iters = n_tiles_total + kLUQueue + 1;     // no role loops longer than this, whatever it reads

    // Consumers take the tiles in the order the scheduler published them; rows < 0 ends the sequence.
    int q_slot = 0;
    uint32_t q_phase = 0;
    auto next_tile = [&]() {
        if (!timed_out && !ptx::mbar_wait(q_full + q_slot, q_phase)) timed_out = true;
        const Tile tl = queue[q_slot];
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(q_empty + q_slot);
        if (++q_slot == kLUQueue) { q_slot = 0; q_phase ^= 1; }
        return tl;
    };

    if (warp == kLUSchedWarp) {
        // ------------------------------------------------------------------ scheduler
        int fetched = 0;
        int published = 0;
        Tile last;
        last.bin = 0; last.start = 0; last.rows = -1; last.pad = 0;
        // direct lists: tiles of this lane's bins, and of all lanes before it
        const int per_lane = (n_bins + 31) >> 5;
        const int bin0 = min(lane * per_lane, n_bins), bin1 = min(bin0 + per_lane, n_bins);
        int tiles_incl = 0, tiles_mine = 0, tiles_all = 0;
        // (the counts are read with ordinary loads, so that the repeated walks below hit in L1; nothing writes them
        // while any CTA still reads them)
        const bool vec4 = (per_lane & 3) == 0;               // whole 16-byte groups of counts per lane
        if (slot_counts) {
            if (vec4) {
                for (int b = bin0; b < bin1; b += 4) {
                    const int4 c4 = *reinterpret_cast<const int4*>(slot_counts + b);
                    tiles_mine += (c4.x + kLUM - 1) / kLUM + (c4.y + kLUM - 1) / kLUM + (c4.z + kLUM - 1) / kLUM + (c4.w + kLUM - 1) / kLUM;
                }
            } else {
                for (int b = bin0; b < bin1; ++b) tiles_mine += (slot_counts[b] + kLUM - 1) / kLUM;
            }
            tiles_incl = tiles_mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(kFullMask, tiles_incl, o);
                if (lane >= o) tiles_incl += v;
            }
            tiles_all = __shfl_sync(kFullMask, tiles_incl, 31);
        }
        for (;;) {
            // tile n >= 2 is claimed once the gathers have started tile n - 1
            if (published >= 2 && !timed_out && !ptx::mbar_wait_relaxed(want, (uint32_t)(published - 1) & 1u)) timed_out = true;
            int idx = 0;
            if (lane == 0) idx = atomicAdd(sched, 1);
            idx = __shfl_sync(kFullMask, idx, 0);
            Tile c;
            if (slot_counts) {
                if (idx >= tiles_all || ++fetched > max_iters) break;
                int bin = 0, start = 0, rows = 0;
                if (idx >= tiles_incl - tiles_mine && idx < tiles_incl) {       // exactly one lane
                    int rem = idx - (tiles_incl - tiles_mine);
                    // branch-free walk over this lane's bins (the loads do not depend on the running search)
                    auto visit = [&](int b, int cnt) {
                        const int t = (cnt + kLUM - 1) / kLUM;
                        if (rows == 0 && rem < t) {
                            bin = b;
                            start = b * cap + rem * kLUM;
                            rows = min(kLUM, cnt - rem * kLUM);
                        }
                        rem -= t;
                    };
                    if (vec4) {
#pragma unroll 4
                        for (int b = bin0; b < bin1; b += 4) {
                            const int4 c4 = *reinterpret_cast<const int4*>(slot_counts + b);
                            visit(b, c4.x); visit(b + 1, c4.y); visit(b + 2, c4.z); visit(b + 3, c4.w);
                        }
                    } else {
                        for (int b = bin0; b < bin1; ++b) visit(b, slot_counts[b]);
                    }
                }
                const unsigned owner = __ballot_sync(kFullMask, rows > 0);
                if (owner == 0) continue;
                const int src = __ffs(owner) - 1;
                c.bin = __shfl_sync(kFullMask, bin, src);
                c.start = __shfl_sync(kFullMask, start, src);
                c.rows = __shfl_sync(kFullMask, rows, src);
                c.pad = 0;
            } else {
            if (idx >= passes * n_tiles_total || ++fetched > passes * max_iters) break;
            // with two passes the full tiles go first and the ragged ones last, so that the work handed out
            // at the end comes in small pieces
            const int second = idx >= n_tiles_total ? 1 : 0;
            c = tiles[idx - second * n_tiles_total];
            }
            if (c.rows <= 0 || c.rows > kLUM) continue;          // empty list entry
            if (!slot_counts && passes == 2 && (c.rows == kLUM) != (idx < n_tiles_total)) continue;
            if (!timed_out && !ptx::mbar_wait_relaxed(q_empty + q_slot, q_phase ^ 1)) timed_out = true;
            if (lane == 0) {
                queue[q_slot] = c;
                ptx::mbar_arrive(q_full + q_slot);
            }
            __syncwarp();
            if (++q_slot == kLUQueue) { q_slot = 0; q_phase ^= 1; }
            ++published;
        }
        // end of the sequence; after a timeout every slot gets the marker so that stragglers stop too
        for (int s = 0; s < (timed_out ? kLUQueue : 1); ++s) {
            if (!timed_out && !ptx::mbar_wait_relaxed(q_empty + q_slot, q_phase ^ 1)) timed_out = true;
            if (lane == 0) {
                queue[q_slot] = last;
                ptx::mbar_arrive(q_full + q_slot);
            }
            __syncwarp();
            if (++q_slot == kLUQueue) { q_slot = 0; q_phase ^= 1; }
        }
    } else if (warp >= kLUFirstGatherWarp) {
        // ------------------------------------------------------------------ row gathers
        const int gw = warp - kLUFirstGatherWarp;
        int stage = 0;
        uint32_t phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Tile tl = next_tile();
            if (tl.rows <= 0) break;
            if (gw == 0 && lane == 0) ptx::mbar_arrive(want);
            // 4-row group g = lane * kLUGatherWarps + gw of the tile belongs to this lane
            const int total_groups = (tl.rows + 3) >> 2;
            const int groups = max((total_groups - gw + kLUGatherWarps - 1) / kLUGatherWarps, 0);     // of this warp
            const int first = (lane * kLUGatherWarps + gw) * 4;
            int r[4] = {0, 0, 0, 0};
            if (lane < groups) {
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = perm[tl.start + min(first + i, tl.rows - 1)];
            }
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                if (lane == 0) {
                    const uint32_t bytes = (uint32_t)groups * (512u * L::kSub) + (gw == 0 ? (uint32_t)L::kW1CopyBytes : 0u);
                    if (bytes > 0) ptx::mbar_arrive_expect_tx(full + stage, bytes);
                    else ptx::mbar_arrive(full + stage);
                    if (gw == 0) {
                        if constexpr (kW8)
                            ptx::bulk_g2s(ring + stage * L::kStageBytes + L::kXStageBytes + L::kW1StageBytes,
                                          w1codes + ((int64_t)tl.bin * KB + kb) * L::kW1CodeBytes, L::kW1CodeBytes, full + stage);
                        else
                            ptx::bulk_g2s(ring + stage * L::kStageBytes + L::kXStageBytes,
                                          w1img + ((int64_t)tl.bin * KB + kb) * (L::kW1StageBytes / 2), L::kW1StageBytes, full + stage);
                    }
                }
                __syncwarp();
                if (lane < groups) {
#pragma unroll
                    for (int sb = 0; sb < L::kSub; ++sb)
                        ptx::tma_gather4(ring + stage * L::kStageBytes + sb * L::kXSubBytes + first * 128, &tmap_x,
                                         (kb * L::kSub + sb) * kLUKB, r[0], r[1], r[2], r[3], full + stage);
                }
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == kLUGemm1Warp) {
        // ------------------------------------------------------------------ GEMM1 issuer
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(kLUM, L::kN1);
        int stage = 0;
        uint32_t phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Tile tl = next_tile();
            if (tl.rows <= 0) break;
            if (!timed_out && !ptx::mbar_wait(acc1_empty, (it & 1) ^ 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                ptx::tc_fence_after_sync();
                if constexpr (kW8) {
                    // the stage's W1 codes -> bf16 operand tiles (kSub tiles of LP rows x 64 columns, stacked)
                    unsigned char* w1s = ring + stage * L::kStageBytes + L::kXStageBytes;
                    expand_e4m3_tile<kLUKB>(w1s + L::kW1StageBytes, w1s, L::kSub * LP, lane);
                    ptx::fence_proxy_async();
                    __syncwarp();
                }
                if (lane == 0) {
                    const uint32_t xs = ptx::smem_addr(ring + stage * L::kStageBytes);
#pragma unroll
                    for (int sb = 0; sb < L::kSub; ++sb) {
                        const uint64_t ad = ptx::umma_desc_k128(xs + sb * L::kXSubBytes);
                        const uint64_t bd = ptx::umma_desc_k128(xs + L::kXStageBytes + sb * L::kW1SubBytes);
#pragma unroll
                        for (int j = 0; j < kLUKB / 16; ++j)
                            ptx::umma_bf16(tmem_base, ad + 2 * j, bd + 2 * j, idesc, (kb | sb | j) != 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(empty + stage);
                    if (kb == KB - 1) ptx::umma_commit(acc1_full);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == kLUGemm2Warp) {
        // ------------------------------------------------------------------ W2 copies + GEMM2 issuer
        int ld_slot = 0, mm_slot = 0;
        uint32_t ld_phase = 0, mm_phase = 0;
        int pc = 0;                                              // pieces issued so far (selects the accumulator)
        const uint32_t hs = ptx::smem_addr(hbuf);
        for (int it = 0; it < max_iters; ++it) {
            const Tile tl = next_tile();
            if (tl.rows <= 0) break;
            const unsigned char* w2j = w2img + (int64_t)tl.bin * P * L::kW2PieceBytes;
            int loaded = 0;
            // the next piece of this tile into the next ring slot; `block`: wait for the slot, else only if it is free
            auto load_piece = [&](bool block) {
                if (block) {
                    if (!timed_out && !ptx::mbar_wait(w2_empty + ld_slot, ld_phase ^ 1)) timed_out = true;
                } else if (!__any_sync(kFullMask, ptx::mbar_test(w2_empty + ld_slot, ld_phase ^ 1))) {
                    return false;
                }
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(w2_full + ld_slot, (uint32_t)L::kW2PieceBytes);
                    ptx::bulk_g2s(w2ring + ld_slot * L::kW2SlotStride + L::kW2CopyOff, w2j + (int64_t)loaded * L::kW2PieceBytes,
                                  L::kW2PieceBytes, w2_full + ld_slot);
                }
                __syncwarp();
                ++loaded;
                if (++ld_slot == L::kW2Slots) { ld_slot = 0; ld_phase ^= 1; }
                return true;
            };
            // Copies run as far ahead as free slots allow, but only the piece that the next MMA needs is waited for: with
            // fewer slots than pieces (grouped tiles) a wait for the slot of piece p + slots right after the MMA of piece p
            // would hold back the MMA of piece p + 1, whose operands are already there.
            auto load_ahead = [&](int needed) {
                while (loaded < P && load_piece(loaded <= needed)) {}
            };
            load_ahead(-1);
            if (!timed_out && !ptx::mbar_wait(h_full, it & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int p = 0; p < P; ++p, ++pc) {
                const int b = pc & 1;
                load_ahead(p);
                if (!timed_out && !ptx::mbar_wait(w2_full + mm_slot, mm_phase)) timed_out = true;
                if constexpr (kW8) {
                    // the piece's codes -> bf16 operand tile (128 output features x LP columns)
                    unsigned char* slot = w2ring + mm_slot * L::kW2SlotStride;
                    expand_e4m3_tile<LP>(slot + L::kW2CopyOff, slot, kLUPiece, lane);
                    ptx::fence_proxy_async();
                    __syncwarp();
                }
                if (!timed_out && !ptx::mbar_wait(y_empty + b, ((pc >> 1) & 1) ^ 1)) timed_out = true;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const int n = min(kLUPiece, O - p * kLUPiece);
                    const uint32_t idesc = ptx::umma_idesc_bf16(kLUM, n);
                    const uint32_t ws = ptx::smem_addr(w2ring + mm_slot * L::kW2SlotStride);
#pragma unroll
                    for (int blk = 0; blk < L::kHBlocks; ++blk) {
                        // (one K-block of LP columns, or with grouped tiles K-blocks of 64 columns: [128 rows][128 bytes] each)
                        const uint64_t ad = ptx::umma_desc_rows(hs + blk * (kLUM * L::kRowBytes), L::kRowBytes);
                        const uint64_t bd = ptx::umma_desc_rows(ws + blk * (kLUPiece * L::kRowBytes), L::kRowBytes);
#pragma unroll
                        for (int kk = 0; kk < L::kRowBytes / 32; ++kk)
                            ptx::umma_bf16(tmem_base + L::kAcc2Col + b * kLUAccStride, ad + 2 * kk, bd + 2 * kk, idesc,
                                           (blk | kk) != 0 ? 1u : 0u);
                    }
                    ptx::umma_commit(w2_empty + mm_slot);
                    ptx::umma_commit(y_full + b);
                }
                __syncwarp();
                if (++mm_slot == L::kW2Slots) { mm_slot = 0; mm_phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token row and one column part per thread
        // A warp can only read the 32 tensor-memory lanes of its quarter, so a tile of at most 32 (64) rows would
        // leave three quarters (one half) of the epilogue warps without work and cost as much as a full tile.
        // Short tiles are therefore stacked `rep` = 4 (2) times in the 128 rows of GEMM2: H row r is written to the
        // rows r, r + 128/rep, ... of the A operand, every copy's accumulator rows then hold the same values (the
        // rows of an MMA are independent; the extra MMA rows cost nothing), and the quarters of copy c convert and
        // store only the c-th group of 128/rep columns of each piece.
        const int quarter = warp & 3, part = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        constexpr int HC = LP / kLUHParts;                       // H columns of a thread that computes H
        int pc = 0;
        int w2_slot = 0;
        uint32_t w2_phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Tile tl = next_tile();
            if (tl.rows <= 0) break;
            const int rep = GL > 1 ? 1 : tl.rows <= 32 ? 4 : tl.rows <= 64 ? 2 : 1;      // (grouped tiles are not stacked)
            const int qper = 4 / rep;                            // lane quarters per copy
            const int copy = quarter / qper;                     // the copy this thread's lanes hold = its column group
            const int row = (quarter % qper) * 32 + lane;        // the token row this thread's lane carries
            const bool active = (quarter % qper) * 32 < tl.rows; // this warp's lanes hold valid rows
            const bool h_active = active && copy == 0 && part < kLUHParts;      // the first copy's lanes hold acc1
            const int64_t tok = row < tl.rows ? perm[tl.start + row] : -1;
            // accumulator -> pre-activation / output: + bias, and with 8-bit weights the leaf's scale first
            float s1 = 1.0f, s2 = 1.0f;
            if constexpr (kW8) {
                s1 = __ldg(scale1 + tl.bin);
                s2 = __ldg(scale2 + tl.bin);
            }
            auto scaled = [](uint32_t acc, float scale, float bias) {
                if constexpr (kW8) return fmaf(__uint_as_float(acc), scale, bias);
                else return __uint_as_float(acc) + bias;
            };
            if constexpr (GL == 1) {
                float b1r[HC];
#pragma unroll
                for (int j = 0; j < HC; j += 4) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(b1img + (int64_t)tl.bin * LP + (part % kLUHParts) * HC + j));
                    b1r[j] = t.x; b1r[j + 1] = t.y; b1r[j + 2] = t.z; b1r[j + 3] = t.w;
                }

                // H = act(acc1 + b1) -> bf16 -> this thread's part of its row of the A operand of GEMM2 (every copy of it)
                if (!timed_out && !ptx::mbar_wait(acc1_full, it & 1)) timed_out = true;
                ptx::tc_fence_after_sync();
                {
                    uint32_t hp[HC / 2];
                    if (h_active) {
                        uint32_t v[32];
                        ptx::tmem_ld32(lane_base + part * HC, v);      // columns past HC are not used
                        ptx::tmem_ld_wait();
                        with_activation(act, [&](auto a) {
                            constexpr int kAct = decltype(a)::value;
#pragma unroll
                            for (int j = 0; j < HC; j += 2) {
                                float h0 = activate_bf16(kAct, scaled(v[j], s1, b1r[j]));
                                float h1 = activate_bf16(kAct, scaled(v[j + 1], s1, b1r[j + 1]));
                                if (kFold && part * HC + j == l) h0 = 1.0f;          // the bias column
                                if (kFold && part * HC + j + 1 == l) h1 = 1.0f;
                                hp[j / 2] = ptx::pack_bf16(h0, h1);
                            }
                        });
                    }
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive(acc1_empty);
                    if (h_active) {
                        for (int cp = 0; cp < rep; ++cp) {
                            const int hrow = row + cp * (kLUM / rep);
#pragma unroll
                            for (int c = 0; c < HC / 8; ++c)
                                *reinterpret_cast<uint4*>(hbuf + swz_rows((uint32_t)(hrow * L::kRowBytes + (part * HC / 8 + c) * 16), L::kRowBytes)) =
                                    make_uint4(hp[4 * c], hp[4 * c + 1], hp[4 * c + 2], hp[4 * c + 3]);
                        }
                        ptx::fence_proxy_async();
                    }
                    ptx::mbar_arrive(h_full);
                }
            } else {
                // Grouped tile: the row's leaf first (three levels from the subtree's 7 node logits, accumulator columns
                // 8 LP ..), then H = act(acc1 + b1) for that leaf's LP columns; the row's other 7 LP columns of the
                // A operand of GEMM2 are zero.  Both column parts walk (the walk is cheap); part p writes K-block p of the
                // row (the columns of leaves 4p .. 4p + 3).
                const float* gb = g1bias + (int64_t)tl.bin * L::kN1;
                float nb[8];
                {
                    const float4 q0 = __ldg(reinterpret_cast<const float4*>(gb + GL * LP));
                    const float4 q1 = __ldg(reinterpret_cast<const float4*>(gb + GL * LP + 4));
                    nb[0] = q0.x; nb[1] = q0.y; nb[2] = q0.z; nb[3] = q0.w; nb[4] = q1.x; nb[5] = q1.y; nb[6] = q1.z; nb[7] = q1.w;
                }
                if (!timed_out && !ptx::mbar_wait(acc1_full, it & 1)) timed_out = true;
                ptx::tc_fence_after_sync();
                int j = 0;                                   // the row's leaf among the 8
                float pre[LP];
                if (active) {
                    uint32_t nv[16];
                    ptx::tmem_ld16(lane_base + GL * LP, nv);
                    ptx::tmem_ld_wait();
                    // a logit of zero goes right, NaN left (as in the descent kernels)
                    const int n0 = __uint_as_float(nv[0]) + nb[0] >= 0.0f ? 1 : 0;
                    const float l1 = n0 ? __uint_as_float(nv[2]) + nb[2] : __uint_as_float(nv[1]) + nb[1];
                    const int q = 2 * n0 + (l1 >= 0.0f ? 1 : 0);
                    const float l2 = q == 0 ? __uint_as_float(nv[3]) + nb[3] : q == 1 ? __uint_as_float(nv[4]) + nb[4]
                                   : q == 2 ? __uint_as_float(nv[5]) + nb[5] : __uint_as_float(nv[6]) + nb[6];
                    j = 2 * q + (l2 >= 0.0f ? 1 : 0);
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc) {
                        uint32_t v[32];
                        ptx::tmem_ld32(lane_base + part * 64 + cc * 32, v);
                        ptx::tmem_ld_wait();
                        if (((j & 3) >> 1) == cc) {
#pragma unroll
                            for (int i = 0; i < LP; ++i) pre[i] = __uint_as_float((j & 1) ? v[LP + i] : v[i]);
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(acc1_empty);
                if (active) {
                    const bool own = (j >> 2) == part;
                    uint32_t hp[LP / 2];
#pragma unroll
                    for (int i = 0; i < LP / 2; ++i) hp[i] = 0u;
                    if (own) {
                        float b1r[LP];
#pragma unroll
                        for (int i = 0; i < LP; i += 4) {
                            const float4 t = __ldg(reinterpret_cast<const float4*>(gb + j * LP + i));
                            b1r[i] = t.x; b1r[i + 1] = t.y; b1r[i + 2] = t.z; b1r[i + 3] = t.w;
                        }
                        with_activation(act, [&](auto a) {
                            constexpr int kAct = decltype(a)::value;
#pragma unroll
                            for (int i = 0; i < LP; i += 2) {
                                float h0 = activate_bf16(kAct, pre[i] + b1r[i]);
                                float h1 = activate_bf16(kAct, pre[i + 1] + b1r[i + 1]);
                                if (i == l) h0 = 1.0f;                           // the bias column
                                if (i + 1 == l) h1 = 1.0f;
                                hp[i / 2] = ptx::pack_bf16(h0, h1);
                            }
                        });
                    }
                    // the row's 128 bytes of K-block `part`: the leaf's two 16-byte units, zeros elsewhere
                    const int du = own ? (j & 3) * (LP / 8) : -8;
                    unsigned char* hb = hbuf + part * (kLUM * L::kRowBytes);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        uint4 val = make_uint4(0u, 0u, 0u, 0u);
                        if (u == du) val = make_uint4(hp[0], hp[1], hp[2], hp[3]);
                        if (u == du + 1) val = make_uint4(hp[4], hp[5], hp[6], hp[7]);
                        *reinterpret_cast<uint4*>(hb + swz_rows((uint32_t)(row * L::kRowBytes + u * 16), L::kRowBytes)) = val;
                    }
                    ptx::fence_proxy_async();
                    if (part == 0 && tok >= 0) {
                        const int32_t leaf = tl.bin * GL + j;
                        if (leaf_out) leaf_out[tok] = leaf;
                        if (leaf_out2) leaf_out2[tok] = leaf;
                    }
                }
                ptx::mbar_arrive(h_full);
            }

            // Y pieces: this thread's share of the 128 columns: 64 / rep columns of column group `copy`
            __nv_bfloat16* yrow = y + (tok >= 0 ? tok : 0) * O;
            const int ncw = (kLUPiece / kLUColParts) / rep;          // 64, 32 or 16
            const int cbase = copy * (kLUPiece / rep) + part * ncw;
            for (int p = 0; p < P; ++p, ++pc) {
                const int b = pc & 1;
                if (!timed_out && !ptx::mbar_wait(y_full + b, (pc >> 1) & 1)) timed_out = true;
                if (!timed_out && !ptx::mbar_wait(w2_full + w2_slot, w2_phase)) timed_out = true;     // biases: landed long ago
                ptx::tc_fence_after_sync();
                const float* bias = reinterpret_cast<const float*>(w2ring + w2_slot * L::kW2SlotStride + L::kW2BiasOff);
                const int ncols = min(kLUPiece, O - p * kLUPiece);
                if (ncw == 16) {
                    const int c0 = cbase;
                    if (active && c0 < ncols) {                      // ncols is a multiple of 16
                        uint32_t v[16];
                        ptx::tmem_ld16(lane_base + L::kAcc2Col + b * kLUAccStride + c0, v);
                        ptx::tmem_ld_wait();
                        uint32_t out[8];
                        if (kFold) {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                out[e] = ptx::pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float4 bb = *reinterpret_cast<const float4*>(bias + c0 + 4 * e);
                                out[2 * e] = ptx::pack_bf16(scaled(v[4 * e], s2, bb.x), scaled(v[4 * e + 1], s2, bb.y));
                                out[2 * e + 1] = ptx::pack_bf16(scaled(v[4 * e + 2], s2, bb.z), scaled(v[4 * e + 3], s2, bb.w));
                            }
                        }
                        if (tok >= 0) {
                            const int o0 = p * kLUPiece + c0;
                            if (wide_stores) {
                                ptx::st_global_v8(yrow + o0, out);
                            } else {
                                *reinterpret_cast<uint4*>(yrow + o0) = make_uint4(out[0], out[1], out[2], out[3]);
                                *reinterpret_cast<uint4*>(yrow + o0 + 8) = make_uint4(out[4], out[5], out[6], out[7]);
                            }
                        }
                    }
                } else {
                    for (int cc = 0; cc * 32 < ncw; ++cc) {
                        const int c0 = cbase + cc * 32;
                        const int nv = min(32, ncols - c0);              // <= 0, 16 or 32
                        if (active && nv > 0) {
                            uint32_t v[32];
                            ptx::tmem_ld32(lane_base + L::kAcc2Col + b * kLUAccStride + c0, v);
                            ptx::tmem_ld_wait();
                            const int o0 = p * kLUPiece + c0;
                            uint32_t out[16];
                            if (kFold) {                                 // bias already added by GEMM2
#pragma unroll
                                for (int e = 0; e < 16; ++e)
                                    out[e] = ptx::pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
                            } else {
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const float4 bb = *reinterpret_cast<const float4*>(bias + c0 + 4 * e);
                                    out[2 * e] = ptx::pack_bf16(scaled(v[4 * e], s2, bb.x), scaled(v[4 * e + 1], s2, bb.y));
                                    out[2 * e + 1] = ptx::pack_bf16(scaled(v[4 * e + 2], s2, bb.z), scaled(v[4 * e + 3], s2, bb.w));
                                }
                            }
                            if (tok >= 0) {
                                if (wide_stores && nv == 32) {
                                    ptx::st_global_v8(yrow + o0, out);
                                    ptx::st_global_v8(yrow + o0 + 16, out + 8);
                                } else {
#pragma unroll
                                    for (int q = 0; q < 4; ++q)
                                        if (q * 8 < nv)
                                            *reinterpret_cast<uint4*>(yrow + o0 + q * 8) =
                                                make_uint4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
                                }
                            }
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(y_empty + b);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(w2_empty + w2_slot);
                if (++w2_slot == L::kW2Slots) { w2_slot = 0; w2_phase ^= 1; }
            }
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let copies and MMAs still in flight finish before exit
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kLUGemm1Warp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kLUTmemCols);
    }
    // the last CTA to finish rearms the scheduler words (and the direct lists' counts) for the next launch
    if (warp == 0) {
        int is_last = 0;
        if (lane == 0) {
            __threadfence();
            is_last = atomicAdd(sched + 1, 1) == (int)gridDim.x - 1 ? 1 : 0;
        }
        is_last = __shfl_sync(kFullMask, is_last, 0);
        if (is_last) {
            if (slot_counts)
                for (int b = lane; b < n_bins; b += 32) slot_counts[b] = 0;
            if (lane == 0) {
                sched[0] = 0;
                sched[1] = 0;
            }
            __threadfence();
        }
    }
}

}  // namespace fff
