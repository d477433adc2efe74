// Grouped leaf evaluation on tcgen05 for thin buckets: G buckets share the 128 rows of one tcgen05.mma.
//
// Algorithm 1, FORWARD_I, leaf branch, as in leaf_umma.cuh.  There a tile is up to 128 tokens of one leaf;
// with a few dozen tokens per leaf most accumulator rows are idle, yet the epilogue (which can only be
// spread over rows: a warp reads the 32 tensor-memory lanes of its own quarter) takes as long as for a
// full tile.  Here a work unit is a group of G = 2 or 4 sub-tiles of up to R = 128 / G tokens, each of its
// own leaf, stacked in the rows of one operand tile (sub-tile q = rows q R .. q R + R - 1):
//   GEMM1  per K-block and sub-tile q one MMA group  acc1[:, q LP .. q LP + LP) = X W1_q^T  over all 128
//          rows; a row only ever reads the column block of its own sub-tile, the others are by-products;
//          two accumulators, so that the loads of the next group never wait for the epilogue of this one;
//   H      G operand buffers; the rows of sub-tile q are written to buffer q only, all other rows of
//          buffer q are zero from the start of the kernel and stay zero;
//   GEMM2  per piece  acc2 = sum_q H_q W2_q^T: the zero rows make every row see its own leaf's W2 alone;
//          the output bias rides in GEMM2 (l < LP, see leaf_umma.cuh) or is added per row in the epilogue.
// The extra MMAs are free (the tensor pipe is a few per cent busy in this memory-bound step); weight
// images, roles, barriers, the just-in-time tile scheduler and the bounded waits are those of k_leaf_umma.
// 0 x Inf is NaN: a leaf with non-finite W2 entries would reach the rows of its group mates through the
// zero rows, so the host takes this kernel only when every W2 and b2 entry is finite.
//
// Requirements: as k_leaf_umma; the tile list is made for R-row tiles and read in groups of G entries.
#pragma once

#include "leaf_umma.cuh"

namespace fff {

template <int G> struct TileGroup {
    Tile t[G];
};

constexpr int kLPAcc2Col = 256;            // first tensor-memory column of the two GEMM2 accumulators

template <int LP, int G> struct LeafPackLayout {
    static_assert(LP == 16 || LP == 32 || LP == 64, "padded hidden width");
    static_assert(G == 2 || G == 4, "sub-tiles per group");
    static constexpr int kSubRows = kLUM / G;
    static constexpr int kQuartersPerSub = kSubRows / 32;
    static constexpr int kRowBytes = LP * 2;
    // K-blocks of 64 columns per ring stage.  Two per stage (with three stages and a smaller W2 ring) measured the
    // same; a W2 ring below 72 KB measured slower.
    static constexpr int kSub = 1;
    static constexpr int kXSubBytes = kLUM * kLUKB * 2;                      // one K-block of the token rows
    static constexpr int kW1SubBytes = LP * kLUKB * 2;                       // one leaf's K-block of W1
    static constexpr int kXStageBytes = kSub * kXSubBytes;
    static constexpr int kW1Bytes = kSub * kW1SubBytes;                      // one leaf's share of a stage
    static constexpr int kStageBytes = kXStageBytes + G * kW1Bytes;          // a multiple of 1024
    static constexpr int kW2Bytes = kLUPiece * kRowBytes;
    static constexpr int kW2PieceBytes = kW2Bytes + kLUPiece * 4;            // + float32 biases
    static constexpr int kW2SubStride = (kW2PieceBytes + 1023) & ~1023;
    static constexpr int kW2SlotStride = G * kW2SubStride;                   // a piece of every sub-tile's leaf
    static constexpr int kW2Want = 72 * 1024 / kW2SlotStride;
    static constexpr int kW2Slots = kW2Want < 2 ? 2 : kW2Want > 8 ? 8 : kW2Want;
    static constexpr int kHBytes = kLUM * kRowBytes;                         // one of the G buffers
    static constexpr int kBarrierBytes = 1024;
    static constexpr int kAcc1Cols = G * LP;                                 // of one of the two GEMM1 accumulators
    static_assert(2 * kAcc1Cols <= kLPAcc2Col, "GEMM1 accumulator columns");
    static constexpr int smem_bytes(int stages) {
        return 1024 + stages * kStageBytes + kW2Slots * kW2SlotStride + G * kHBytes + kBarrierBytes;
    }
};

// sched: as for k_leaf_umma ([0] groups handed out, [1] CTAs finished; zero before and after every launch).
template <int LP, bool kFold, int G>
__global__ void __launch_bounds__(kLUThreads, 1)
k_leaf_umma_packed(const __grid_constant__ CUtensorMap tmap_x, const int32_t* __restrict__ perm,
                   const Tile* __restrict__ tiles, int n_tiles_total,
                   const __nv_bfloat16* __restrict__ w1img, const float* __restrict__ b1img,
                   const unsigned char* __restrict__ w2img, __nv_bfloat16* __restrict__ y,
                   int D, int O, int l, int act, int kStages, int wide_stores, int* __restrict__ sched,
                   int* __restrict__ status)
{
    using L = LeafPackLayout<LP, G>;
    using Group = TileGroup<G>;
    constexpr int R = L::kSubRows;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* w2ring = ring + kStages * L::kStageBytes;
    unsigned char* hbuf = w2ring + L::kW2Slots * L::kW2SlotStride;
    uint64_t* full = reinterpret_cast<uint64_t*>(hbuf + G * L::kHBytes);
    uint64_t* empty = full + kLUMaxStages;
    uint64_t* w2_full = empty + kLUMaxStages;
    uint64_t* w2_empty = w2_full + kLUMaxW2Slots;
    uint64_t* q_full = w2_empty + kLUMaxW2Slots;
    uint64_t* q_empty = q_full + kLUQueue;
    uint64_t* acc1_full = q_empty + kLUQueue;      // [2]
    uint64_t* acc1_empty = acc1_full + 2;          // [2]
    uint64_t* h_full = acc1_empty + 2;
    uint64_t* y_full = h_full + 1;          // [2]
    uint64_t* y_empty = y_full + 2;         // [2]
    uint64_t* want = y_empty + 2;           // the gathers have started another group
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(want + 1);
    Group* queue = reinterpret_cast<Group*>(tmem_slot + 2);                  // [kLUQueue]
    static_assert((8 + 8 + 12 + 12 + 4 + 4 + 2 + 2 + 1 + 2 + 2 + 1) * 8 + 8 + kLUQueue * (int)sizeof(Group) <= L::kBarrierBytes,
                  "barrier area");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = D / (kLUKB * L::kSub);                    // ring stages per group
    const int P = (O + kLUPiece - 1) / kLUPiece;
    const int n_groups = (n_tiles_total + G - 1) / G;

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
        ptx::mbar_init(h_full, kLUEpiWarps * 32);
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(acc1_full + b, 1);
            ptx::mbar_init(acc1_empty + b, kLUEpiWarps * 32);
            ptx::mbar_init(y_full + b, 1);
            ptx::mbar_init(y_empty + b, kLUEpiWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    // the H buffers start out zero; only the rows of a buffer's own sub-tile are ever written
    for (int i = threadIdx.x; i < G * L::kHBytes / 16; i += kLUThreads) reinterpret_cast<uint4*>(hbuf)[i] = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async();
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
    const int max_iters = n_groups + kLUQueue + 1;          // no role loops longer than this, whatever it reads

    // Consumers take the groups in the order the scheduler published them; t[0].rows < 0 ends the sequence.
    int q_slot = 0;
    uint32_t q_phase = 0;
    auto next_group = [&]() {
        if (!timed_out && !ptx::mbar_wait(q_full + q_slot, q_phase)) timed_out = true;
        const Group g = queue[q_slot];
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(q_empty + q_slot);
        if (++q_slot == kLUQueue) { q_slot = 0; q_phase ^= 1; }
        return g;
    };

    if (warp == kLUSchedWarp) {
        // ------------------------------------------------------------------ scheduler
        int fetched = 0;
        int published = 0;
        for (;;) {
            // group n >= 2 is claimed once the gathers have started group n - 1
            if (published >= 2 && !timed_out && !ptx::mbar_wait_relaxed(want, (uint32_t)(published - 1) & 1u)) timed_out = true;
            int idx = 0;
            if (lane == 0) idx = atomicAdd(sched, 1);
            idx = __shfl_sync(kFullMask, idx, 0);
            if (idx >= n_groups || ++fetched > max_iters) break;
            Group c;
            bool any = false;
#pragma unroll
            for (int q = 0; q < G; ++q) {
                const int li = idx * G + q;
                Tile t;
                t.bin = 0; t.start = 0; t.rows = 0; t.pad = 0;
                if (li < n_tiles_total) t = tiles[li];
                if (t.rows <= 0 || t.rows > R) { t.bin = 0; t.start = 0; t.rows = 0; }     // empty list entry
                else any = true;
                c.t[q] = t;
            }
            if (!any) continue;
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
        Group last;
#pragma unroll
        for (int q = 0; q < G; ++q) { last.t[q].bin = 0; last.t[q].start = 0; last.t[q].rows = -1; last.t[q].pad = 0; }
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
        // ------------------------------------------------------------------ row gathers + W1 K-blocks
        const int gw = warp - kLUFirstGatherWarp;
        // lanes 0-7: the 4-row group lane * 4 + gw of the operand tile
        const int srow = ((lane & 7) * kLUGatherWarps + gw) * 4;             // its first operand row
        const int sub = srow / R, r0 = srow - sub * R;
        int stage = 0;
        uint32_t phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Group g = next_group();
            if (g.t[0].rows < 0) break;
            if (gw == 0 && lane == 0) ptx::mbar_arrive(want);
            Tile mine = g.t[0];
#pragma unroll
            for (int q = 1; q < G; ++q)
                if (q == sub) mine = g.t[q];
            const bool valid = lane < 8 && r0 < mine.rows;
            int r[4] = {0, 0, 0, 0};
            if (valid) {
#pragma unroll
                for (int i = 0; i < 4; ++i) r[i] = perm[mine.start + min(r0 + i, mine.rows - 1)];
            }
            const int n_valid = __popc(__ballot_sync(kFullMask, valid));
            // the W1 K-blocks of sub-tile gw come with this warp's rows
            Tile wt = g.t[0];
#pragma unroll
            for (int q = 1; q < G; ++q)
                if (q == gw) wt = g.t[q];
            const bool w1_mine = gw < G && wt.rows > 0;
            const __nv_bfloat16* w1j = w1img + (int64_t)wt.bin * KB * (L::kSub * LP * kLUKB);
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                unsigned char* st = ring + stage * L::kStageBytes;
                if (lane == 0) {
                    const uint32_t bytes = (uint32_t)n_valid * (512u * L::kSub) + (w1_mine ? (uint32_t)L::kW1Bytes : 0u);
                    if (bytes > 0) ptx::mbar_arrive_expect_tx(full + stage, bytes);
                    else ptx::mbar_arrive(full + stage);
                    if (w1_mine)
                        ptx::bulk_g2s(st + L::kXStageBytes + gw * L::kW1Bytes, w1j + (int64_t)kb * (L::kSub * LP * kLUKB), L::kW1Bytes, full + stage);
                }
                __syncwarp();
                if (valid) {
#pragma unroll
                    for (int sb = 0; sb < L::kSub; ++sb)
                        ptx::tma_gather4(st + sb * L::kXSubBytes + srow * 128, &tmap_x, (kb * L::kSub + sb) * kLUKB, r[0], r[1], r[2], r[3],
                                         full + stage);
                }
                if (++stage == kStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == kLUGemm1Warp) {
        // ------------------------------------------------------------------ GEMM1 issuer
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(kLUM, LP);
        int stage = 0;
        uint32_t phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Group g = next_group();
            if (g.t[0].rows < 0) break;
            const int a = it & 1;                                // GEMM1 accumulator of this group
            if (!timed_out && !ptx::mbar_wait(acc1_empty + a, ((it >> 1) & 1) ^ 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait(full + stage, phase)) timed_out = true;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t xs = ptx::smem_addr(ring + stage * L::kStageBytes);
#pragma unroll
                    for (int q = 0; q < G; ++q) {
                        if (g.t[q].rows <= 0) continue;
#pragma unroll
                        for (int sb = 0; sb < L::kSub; ++sb) {
                            const uint64_t ad = ptx::umma_desc_k128(xs + sb * L::kXSubBytes);
                            const uint64_t bd = ptx::umma_desc_k128(xs + L::kXStageBytes + q * L::kW1Bytes + sb * L::kW1SubBytes);
#pragma unroll
                            for (int j = 0; j < kLUKB / 16; ++j)
                                ptx::umma_bf16(tmem_base + a * L::kAcc1Cols + q * LP, ad + 2 * j, bd + 2 * j, idesc, (kb | sb | j) != 0 ? 1u : 0u);
                        }
                    }
                    ptx::umma_commit(empty + stage);
                    if (kb == KB - 1) ptx::umma_commit(acc1_full + a);
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
            const Group g = next_group();
            if (g.t[0].rows < 0) break;
            int n_act = 0;
#pragma unroll
            for (int q = 0; q < G; ++q) n_act += g.t[q].rows > 0 ? 1 : 0;
            int loaded = 0;
            auto load_piece = [&]() {
                if (!timed_out && !ptx::mbar_wait(w2_empty + ld_slot, ld_phase ^ 1)) timed_out = true;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(w2_full + ld_slot, (uint32_t)(n_act * L::kW2PieceBytes));
#pragma unroll
                    for (int q = 0; q < G; ++q)
                        if (g.t[q].rows > 0)
                            ptx::bulk_g2s(w2ring + ld_slot * L::kW2SlotStride + q * L::kW2SubStride,
                                          w2img + ((int64_t)g.t[q].bin * P + loaded) * L::kW2PieceBytes, L::kW2PieceBytes,
                                          w2_full + ld_slot);
                }
                __syncwarp();
                ++loaded;
                if (++ld_slot == L::kW2Slots) { ld_slot = 0; ld_phase ^= 1; }
            };
            while (loaded < P && loaded < L::kW2Slots) load_piece();
            if (!timed_out && !ptx::mbar_wait(h_full, it & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            for (int p = 0; p < P; ++p, ++pc) {
                const int b = pc & 1;
                if (!timed_out && !ptx::mbar_wait(w2_full + mm_slot, mm_phase)) timed_out = true;
                if (!timed_out && !ptx::mbar_wait(y_empty + b, ((pc >> 1) & 1) ^ 1)) timed_out = true;
                ptx::tc_fence_after_sync();
                if (lane == 0) {
                    const int n = min(kLUPiece, O - p * kLUPiece);
                    const uint32_t idesc = ptx::umma_idesc_bf16(kLUM, n);
                    const uint32_t ws = ptx::smem_addr(w2ring + mm_slot * L::kW2SlotStride);
                    uint32_t acc = 0;                            // the first MMA of a piece overwrites the accumulator
#pragma unroll
                    for (int q = 0; q < G; ++q) {
                        if (g.t[q].rows <= 0) continue;
                        const uint64_t ad = ptx::umma_desc_rows(hs + q * L::kHBytes, L::kRowBytes);
                        const uint64_t bd = ptx::umma_desc_rows(ws + q * L::kW2SubStride, L::kRowBytes);
#pragma unroll
                        for (int kk = 0; kk < LP / 16; ++kk) {
                            ptx::umma_bf16(tmem_base + kLPAcc2Col + b * kLUAccStride, ad + 2 * kk, bd + 2 * kk, idesc, acc);
                            acc = 1;
                        }
                    }
                    ptx::umma_commit(w2_empty + mm_slot);
                    ptx::umma_commit(y_full + b);
                }
                __syncwarp();
                if (++mm_slot == L::kW2Slots) { mm_slot = 0; mm_phase ^= 1; }
                if (loaded < P) load_piece();                    // when a group has more pieces than ring slots
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token row and one column part per thread
        const int quarter = warp & 3, part = warp >> 2;
        const int row = quarter * 32 + lane;                     // operand and accumulator row
        const int sub = quarter / L::kQuartersPerSub;            // the sub-tile it belongs to
        const int srow = row - sub * R;                          // and its position there
        const int qrow0 = (quarter % L::kQuartersPerSub) * 32;   // first such position of this warp
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        unsigned char* hsub = hbuf + sub * L::kHBytes;
        constexpr int HC = LP / kLUHParts;                       // H columns of a thread that computes H
        constexpr int YC = kLUPiece / kLUColParts;               // y columns of this thread per piece
        int pc = 0;
        int w2_slot = 0;
        uint32_t w2_phase = 0;
        for (int it = 0; it < max_iters; ++it) {
            const Group g = next_group();
            if (g.t[0].rows < 0) break;
            Tile tl = g.t[0];
#pragma unroll
            for (int q = 1; q < G; ++q)
                if (q == sub) tl = g.t[q];
            const bool active = qrow0 < tl.rows;                 // this warp's lanes hold valid rows
            const bool h_active = active && part < kLUHParts;
            const int64_t tok = srow < tl.rows ? perm[tl.start + srow] : -1;
            float b1r[HC];
#pragma unroll
            for (int j = 0; j < HC; j += 4) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(b1img + (int64_t)tl.bin * LP + (part % kLUHParts) * HC + j));
                b1r[j] = t.x; b1r[j + 1] = t.y; b1r[j + 2] = t.z; b1r[j + 3] = t.w;
            }

            // H = act(acc1 + b1) -> bf16 -> this thread's part of its row of its sub-tile's A operand of GEMM2
            const int a = it & 1;
            if (!timed_out && !ptx::mbar_wait(acc1_full + a, (it >> 1) & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            {
                uint32_t hp[HC / 2];
                if (h_active) {
                    uint32_t v[32];
                    ptx::tmem_ld32(lane_base + a * L::kAcc1Cols + sub * LP + part * HC, v);      // columns past HC are not used
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < HC; j += 2) {
                        float h0 = activate_bf16(act, __uint_as_float(v[j]) + b1r[j]);
                        float h1 = activate_bf16(act, __uint_as_float(v[j + 1]) + b1r[j + 1]);
                        if (kFold && part * HC + j == l) h0 = 1.0f;          // the bias column
                        if (kFold && part * HC + j + 1 == l) h1 = 1.0f;
                        hp[j / 2] = ptx::pack_bf16(h0, h1);
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive(acc1_empty + a);
                if (h_active) {
#pragma unroll
                    for (int c = 0; c < HC / 8; ++c)
                        *reinterpret_cast<uint4*>(hsub + swz_rows((uint32_t)(row * L::kRowBytes + (part * HC / 8 + c) * 16), L::kRowBytes)) =
                            make_uint4(hp[4 * c], hp[4 * c + 1], hp[4 * c + 2], hp[4 * c + 3]);
                    ptx::fence_proxy_async();
                }
                ptx::mbar_arrive(h_full);
            }

            // Y pieces: this thread's share of the 128 columns
            __nv_bfloat16* yrow = y + (tok >= 0 ? tok : 0) * O;
            for (int p = 0; p < P; ++p, ++pc) {
                const int b = pc & 1;
                if (!timed_out && !ptx::mbar_wait(y_full + b, (pc >> 1) & 1)) timed_out = true;
                if (!timed_out && !ptx::mbar_wait(w2_full + w2_slot, w2_phase)) timed_out = true;     // biases: landed long ago
                ptx::tc_fence_after_sync();
                const float* bias = reinterpret_cast<const float*>(w2ring + w2_slot * L::kW2SlotStride + sub * L::kW2SubStride + L::kW2Bytes);
                const int ncols = min(kLUPiece, O - p * kLUPiece);
#pragma unroll
                for (int cc = 0; cc < YC / 32; ++cc) {
                    const int c0 = part * YC + cc * 32;
                    const int nv = min(32, ncols - c0);              // <= 0, 16 or 32
                    if (active && nv > 0) {
                        uint32_t v[32];
                        ptx::tmem_ld32(lane_base + kLPAcc2Col + b * kLUAccStride + c0, v);
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
                                out[2 * e] = ptx::pack_bf16(__uint_as_float(v[4 * e]) + bb.x, __uint_as_float(v[4 * e + 1]) + bb.y);
                                out[2 * e + 1] = ptx::pack_bf16(__uint_as_float(v[4 * e + 2]) + bb.z, __uint_as_float(v[4 * e + 3]) + bb.w);
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
    // the last CTA to finish rearms the scheduler words for the next launch
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace fff
