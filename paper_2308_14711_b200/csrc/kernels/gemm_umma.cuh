// Dense bf16 GEMM on the fifth-generation tensor cores, C = epilogue(A . B^T), for FORWARD_T.
//
// Algorithm 1, FORWARD_T: the training-time forward pass evaluates EVERY node and EVERY leaf for every
// token and mixes the leaf outputs with the products of the node choices along the root paths.  Unlike
// hard inference this is a true dense contraction, so it runs as three GEMMs with fused epilogues:
//   kGemmNodes   c[t, r]   = sigmoid(<x_t, w_r> + b_r)                    for all 2^d - 1 nodes r
//   kGemmHidden  h'[t, q]  = mix[t, leaf(q)] * act(<x_t, W1_q> + b1_q)    for all 2^d l hidden neurons q
//   kGemmOutput  y[t, o]   = sum_q h'[t, q] W2[o, q] + sum_j mix[t, j] b2[j, o]
// (the mixture of the output biases rides in 2^d extra columns of the K dimension of the last GEMM).
//
// A is [M, K] and B is [N, K], both row-major with K contiguous, read through tensor maps (128-byte
// swizzle, rows outside the matrix read as zeros).  One persistent CTA per SM works on 128 x 256 tiles of
// C: one warp issues the tensor-map loads of the K-blocks (64 columns) into a ring of shared-memory stages,
// another issues four tcgen05.mma (M = 128, N = 256, K = 16) per stage into one of two accumulators in
// tensor memory, the others read the finished accumulator (one row per thread), apply the epilogue and
// store (sixteen epilogue warps: four per lane quarter, 64 columns each).  Tiles that share their rows of A are
// neighbours in the schedule, so A is read from DRAM once.
//
// Every wait is bounded (see ptx.cuh); tensor memory is released on every exit path.
// Requirements: bf16, K % 64 == 0, A and B 16-byte aligned with row pitches that are multiples of 16 bytes.
#pragma once

#include <cuda.h>      // CUtensorMap

#include "common.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kGM = 128;                 // rows of C per tile = rows of one tcgen05.mma
constexpr int kGN = 256;                 // columns of C per tile
constexpr int kGKB = 64;                 // K-block: 128 bytes, one swizzle line
constexpr int kGStages = 4;
constexpr int kGEpiWarps = 16;           // four per tensor-memory lane quarter, 64 columns of the tile each: a lone warp per
                                         // scheduler cannot hide the latency of the epilogue arithmetic
constexpr int kGColsPerWarp = kGN / (kGEpiWarps / 4);
constexpr int kGProducerWarp = kGEpiWarps, kGMmaWarp = kGEpiWarps + 1;
constexpr int kGThreads = (kGEpiWarps + 2) * 32;
constexpr int kGStageBytes = (kGM + kGN) * kGKB * 2;                 // 48 KB
constexpr int kGSmemBytes = 1024 + kGStages * kGStageBytes + 256;
constexpr int kGTmemCols = 2 * kGN;

enum : int { kGemmNodes = 0, kGemmHidden = 1, kGemmOutput = 2 };

// Entropy in nats of a Bernoulli choice with probability c, 0 ln 0 = 0.
// (Branch-free: the logarithms take their arguments clamped to the smallest normal float, so that c = 0 and c = 1 give
// 0 x a finite number = 0; with branches the unrolled epilogue would evaluate its 32 values one after the other.)
__device__ __forceinline__ float bernoulli_entropy(float c) {
    const float tiny = 1.17549435e-38f;
    const float d = 1.0f - c;
    return -(c * __logf(fmaxf(c, tiny)) + d * __logf(fmaxf(d, tiny)));
}

struct GemmEpilogueArgs {
    // kGemmNodes: bias = node biases [N] (bf16), out_f32 = c [M, ld_out]; ent_part (optional) = [m tiles * 4][N]
    // sums of the entropies over each warp's 32 rows.
    // kGemmHidden: bias = hidden biases [N] (bf16), mix = [M, n_leaves] float32, l = neurons per leaf,
    // out_bf16 = h' [M, ld_out].
    // kGemmOutput: out_bf16 = y [M, ld_out].
    const __nv_bfloat16* bias;
    const float* mix;
    float* out_f32;
    __nv_bfloat16* out_bf16;
    float* ent_part;
    int ld_out, n_leaves, l, act;
};

template <int MODE>
__global__ void __launch_bounds__(kGThreads, 1)
k_gemm_umma(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, int M, int N, int K,
            GemmEpilogueArgs ep, int* __restrict__ status)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(ring + kGStages * kGStageBytes);
    uint64_t* empty = full + kGStages;
    uint64_t* acc_full = empty + kGStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_mt = (M + kGM - 1) / kGM, n_nt = (N + kGN - 1) / kGN;
    const int n_tiles = n_mt * n_nt;
    const int KB = K / kGKB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGStages; ++s) {
            ptx::mbar_init(full + s, 1);
            ptx::mbar_init(empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full + a, 1);
            ptx::mbar_init(acc_empty + a, kGEpiWarps * 32);
        }
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_b);
    }
    if (warp == kGMmaWarp) {
        ptx::tmem_alloc(tmem_slot, kGTmemCols);
        ptx::tmem_relinquish_alloc_permit();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    bool timed_out = false;
    if (warp == kGProducerWarp) {
        // ------------------------------------------------------------------ producer
        int stage = 0;
        uint32_t phase = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            const int mt = tile / n_nt, nt = tile % n_nt;
            for (int kb = 0; kb < KB; ++kb) {
                if (!timed_out && !ptx::mbar_wait_relaxed(empty + stage, phase ^ 1)) timed_out = true;
                if (lane == 0) {
                    unsigned char* st = ring + stage * kGStageBytes;
                    ptx::mbar_arrive_expect_tx(full + stage, (uint32_t)kGStageBytes);
                    ptx::tma_load_2d(st, &tmap_a, kb * kGKB, mt * kGM, full + stage);
                    ptx::tma_load_2d(st + kGM * kGKB * 2, &tmap_b, kb * kGKB, nt * kGN, full + stage);
                }
                __syncwarp();
                if (++stage == kGStages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == kGMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(kGM, kGN);
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
                    const uint32_t xs = ptx::smem_addr(ring + stage * kGStageBytes);
                    const uint64_t ad = ptx::umma_desc_k128(xs), bd = ptx::umma_desc_k128(xs + kGM * kGKB * 2);
#pragma unroll
                    for (int j = 0; j < kGKB / 16; ++j)
                        ptx::umma_bf16(tmem_base + a * kGN, ad + 2 * j, bd + 2 * j, idesc, (kb | j) != 0 ? 1u : 0u);
                    ptx::umma_commit(empty + stage);
                    if (kb == KB - 1) ptx::umma_commit(acc_full + a);
                }
                __syncwarp();
                if (++stage == kGStages) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one row of C and one quarter of
        // the tile's columns per thread (warps w, w + 4, w + 8, w + 12 share the lanes of quarter w % 4)
        const int quarter = warp & 3, cpart = warp >> 2;
        int it = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
            const int mt = tile / n_nt, nt = tile % n_nt;
            const int a = it & 1;
            const int row = mt * kGM + quarter * 32 + lane;
            const bool row_ok = row < M;
            if (!timed_out && !ptx::mbar_wait(acc_full + a, (it >> 1) & 1)) timed_out = true;
            ptx::tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * kGN;
            for (int c = cpart * (kGColsPerWarp / 32); c < (cpart + 1) * (kGColsPerWarp / 32); ++c) {
                const int col0 = nt * kGN + c * 32;
                if (col0 >= N) break;                                  // warp-uniform
                uint32_t v[32];
                ptx::tmem_ld32(taddr + c * 32, v);
                ptx::tmem_ld_wait();
                const int nv = min(32, N - col0);
                if (MODE == kGemmNodes) {
                    float* out = ep.out_f32 + (int64_t)row * ep.ld_out + col0;
                    float cv[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float logit = __uint_as_float(v[e]) + (e < nv ? __bfloat162float(ep.bias[col0 + e]) : 0.0f);
                        cv[e] = 1.0f / (1.0f + __expf(-logit));
                    }
                    if (row_ok) {
                        if (nv == 32 && (ep.ld_out & 3) == 0) {
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                *reinterpret_cast<float4*>(out + 4 * q) = make_float4(cv[4 * q], cv[4 * q + 1], cv[4 * q + 2], cv[4 * q + 3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (e < nv) out[e] = cv[e];
                        }
                    }
                    if (ep.ent_part) {
                        // sums over the warp's 32 rows of all 32 columns at once: in step s every lane hands one half of
                        // its values to the lane s away and adds what it gets to the half it keeps, so that lane j ends
                        // with the total of column j (31 shuffles instead of 5 per column); the order is fixed
#pragma unroll
                        for (int e = 0; e < 32; ++e) cv[e] = (row_ok && e < nv) ? bernoulli_entropy(cv[e]) : 0.0f;
#pragma unroll
                        for (int sft = 16; sft >= 1; sft >>= 1) {
                            const bool upper = (lane & sft) != 0;
#pragma unroll
                            for (int i = 0; i < sft; ++i) {
                                const float send = upper ? cv[i] : cv[i + sft];
                                const float keep = upper ? cv[i + sft] : cv[i];
                                cv[i] = keep + __shfl_xor_sync(kFullMask, send, sft);
                            }
                        }
                        if (lane < nv) ep.ent_part[((int64_t)mt * 4 + quarter) * N + col0 + lane] = cv[0];
                    }
                } else if (MODE == kGemmHidden) {
                    __nv_bfloat16* out = ep.out_bf16 + (int64_t)row * ep.ld_out + col0;
                    const float* mrow = ep.mix + (int64_t)(row_ok ? row : 0) * ep.n_leaves;
                    uint32_t packed[16];
                    int leaf = col0 / ep.l, u = col0 % ep.l;           // leaf and unit of column col0 + e, stepped along
                    // the mixture weights of the first leaves of the chunk are fetched together, ahead of their use
                    float mpre[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) mpre[q] = leaf + q < ep.n_leaves ? mrow[leaf + q] : 0.0f;
                    // the chunk's 32 biases: four 16-byte loads (col0 is a multiple of 32, the array 16-byte aligned)
                    float bs[32];
                    if (nv == 32) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(ep.bias + col0) + q);
                            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                bs[8 * q + 2 * i] = __uint_as_float(w[i] << 16);
                                bs[8 * q + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
                            }
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) bs[e] = e < nv ? __bfloat162float(ep.bias[col0 + e]) : 0.0f;
                    }
                    with_activation(ep.act, [&](auto a) {
                        constexpr int kAct = decltype(a)::value;
                        if (ep.l >= 11) {
                            // at most four leaves meet in 32 columns: the weight is chosen among the four fetched ones by
                            // selects, and nothing in the loop branches or loads
                            int ahead = 0;
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float h2[2];
#pragma unroll
                                for (int q = 0; q < 2; ++q) {
                                    const float mw = ahead == 0 ? mpre[0] : ahead == 1 ? mpre[1] : ahead == 2 ? mpre[2] : mpre[3];
                                    const float h = mw * activate_bf16(kAct, __uint_as_float(v[e + q]) + bs[e + q]);
                                    h2[q] = e + q < nv ? h : 0.0f;
                                    const bool wrap = ++u == ep.l;
                                    u = wrap ? 0 : u;
                                    ahead += wrap ? 1 : 0;
                                }
                                packed[e / 2] = ptx::pack_bf16(h2[0], h2[1]);
                            }
                        } else {
                            int ahead = 0;
                            float mw = mpre[0];
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float h2[2];
#pragma unroll
                                for (int q = 0; q < 2; ++q) {
                                    const float h = mw * activate_bf16(kAct, __uint_as_float(v[e + q]) + bs[e + q]);
                                    h2[q] = e + q < nv ? h : 0.0f;
                                    if (++u == ep.l) {
                                        u = 0;
                                        ++leaf;
                                        ++ahead;
                                        mw = ahead == 1 ? mpre[1] : ahead == 2 ? mpre[2] : ahead == 3 ? mpre[3]
                                                        : (leaf < ep.n_leaves ? mrow[leaf] : 0.0f);
                                    }
                                }
                                packed[e / 2] = ptx::pack_bf16(h2[0], h2[1]);
                            }
                        }
                    });
                    if (row_ok) {
                        if (nv == 32 && (ep.ld_out & 7) == 0) {
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                *reinterpret_cast<uint4*>(out + q * 8) = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                        } else {
                            for (int e = 0; e < nv; ++e)
                                out[e] = __ushort_as_bfloat16((unsigned short)((packed[e / 2] >> ((e & 1) * 16)) & 0xffffu));
                        }
                    }
                } else {
                    __nv_bfloat16* out = ep.out_bf16 + (int64_t)row * ep.ld_out + col0;
                    uint32_t packed[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) packed[e] = ptx::pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
                    if (row_ok) {
                        if (nv == 32 && (ep.ld_out & 7) == 0) {
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                *reinterpret_cast<uint4*>(out + q * 8) = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                        } else {
                            for (int e = 0; e < nv; ++e)
                                out[e] = __ushort_as_bfloat16((unsigned short)((packed[e / 2] >> ((e & 1) * 16)) & 0xffffu));
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(acc_empty + a);
        }
    }
    if (timed_out) {
        if (lane == 0) atomicExch(status, kDevTimeout);
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let copies and MMAs still in flight finish before exit
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kGMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kGTmemCols);
    }
}

// Mixture weights of FORWARD_T from the node choices: unrolling the recursion of Algorithm 1, leaf j enters the
// output with the product over its root path of c (where the path turns right) or 1 - c (left).
// c: [B, ldc] float32 (node r in column r);  mix: [B, 2^d] float32 (optional: mix_user, a second copy);
// hp_tail: the same weights as bf16 in the last 2^d used columns of the rows of h' (row pitch ld_hp), where
// the output GEMM multiplies them with the output biases; the padding columns up to ld_hp are zeroed.
// The products along the root path of leaf j for kMixTokens tokens at once, for a tree of DEPTH levels (ct[u] = token
// u's node choices, nullptr = no token): all loads are independent of each other and are issued before the products
// start (with a run-time depth the loop stays rolled and every level waits for its own load: DEPTH round trips to L2
// per value, one token at a time).
constexpr int kMixTokens = 4;
template <int DEPTH>
__device__ __forceinline__ void path_products(const float* const (&ct)[kMixTokens], int j, float (&p)[kMixTokens]) {
    float cv[kMixTokens][DEPTH];
#pragma unroll
    for (int u = 0; u < kMixTokens; ++u)
#pragma unroll
        for (int m = 0; m < DEPTH; ++m) cv[u][m] = ct[u] ? ct[u][(1 << m) - 1 + (j >> (DEPTH - m))] : 0.0f;
#pragma unroll
    for (int u = 0; u < kMixTokens; ++u) {
        float q = 1.0f;
#pragma unroll
        for (int m = 0; m < DEPTH; ++m) q *= ((j >> (DEPTH - m - 1)) & 1) ? cv[u][m] : 1.0f - cv[u][m];
        p[u] = q;
    }
}

// Mixture weights of FORWARD_T from the node choices: unrolling the recursion of Algorithm 1, leaf j enters the
// output with the product over its root path of c (where the path turns right) or 1 - c (left).
// c: [B, ldc] float32 (node r in column r);  mix: [B, 2^d] float32 (optional: mix_user, a second copy);
// hp_tail: the same weights as bf16 in the last 2^d used columns of the rows of h' (row pitch ld_hp), where
// the output GEMM multiplies them with the output biases; the padding columns up to ld_hp are zeroed.
// A block takes kMixTokens tokens at a time, a thread one column of each (no 64-bit divisions in the loop).
__global__ void __launch_bounds__(256)
k_mixture_weights(const float* __restrict__ c, int ldc, float* __restrict__ mix, float* __restrict__ mix_user,
                  __nv_bfloat16* __restrict__ hp, int ld_hp, int hidden, int depth, int64_t B)
{
    const int nl = 1 << depth;
    const int tail = ld_hp - hidden;                          // >= nl: mixture columns, then zero padding
    for (int64_t t0 = (int64_t)blockIdx.x * kMixTokens; t0 < B; t0 += (int64_t)gridDim.x * kMixTokens)
    for (int j = threadIdx.x; j < tail; j += blockDim.x) {
        float p[kMixTokens];
#pragma unroll
        for (int u = 0; u < kMixTokens; ++u) p[u] = 0.0f;
        if (j < nl) {
            const float* ct[kMixTokens];
#pragma unroll
            for (int u = 0; u < kMixTokens; ++u) ct[u] = t0 + u < B ? c + (t0 + u) * ldc : nullptr;
            switch (depth) {            // (the same multiplications in the same order in every case)
                case 1: path_products<1>(ct, j, p); break;
                case 2: path_products<2>(ct, j, p); break;
                case 3: path_products<3>(ct, j, p); break;
                case 4: path_products<4>(ct, j, p); break;
                case 5: path_products<5>(ct, j, p); break;
                case 6: path_products<6>(ct, j, p); break;
                case 7: path_products<7>(ct, j, p); break;
                case 8: path_products<8>(ct, j, p); break;
                case 9: path_products<9>(ct, j, p); break;
                case 10: path_products<10>(ct, j, p); break;
                case 11: path_products<11>(ct, j, p); break;
                case 12: path_products<12>(ct, j, p); break;
                default:
#pragma unroll
                    for (int u = 0; u < kMixTokens; ++u) {
                        if (!ct[u]) continue;
                        float q = 1.0f;
                        for (int m = 0; m < depth; ++m) {
                            const float cv = ct[u][(1 << m) - 1 + (j >> (depth - m))];
                            q *= ((j >> (depth - m - 1)) & 1) ? cv : 1.0f - cv;
                        }
                        p[u] = q;
                    }
            }
        }
#pragma unroll
        for (int u = 0; u < kMixTokens; ++u) {
            const int64_t t = t0 + u;
            if (t >= B) break;
            if (j < nl) {
                mix[t * nl + j] = p[u];
                if (mix_user) mix_user[t * nl + j] = p[u];
            }
            hp[t * ld_hp + hidden + j] = __float2bfloat16_rn(p[u]);
        }
    }
}

// Batch means of the node entropies from the per-warp partial sums of the node GEMM, added in a fixed order:
// one warp per node, lane i adds the parts i, i + 32, ... in order, then the lanes' sums are added by a fixed tree.
// Blocks of 8 warps.
__global__ void __launch_bounds__(256)
k_entropy_reduce(const float* __restrict__ part, int n_parts, int n_nodes, int64_t B, float* __restrict__ ent)
{
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= n_nodes) return;
    float s = 0.0f;
    for (int p = lane; p < n_parts; p += 32) s += part[(int64_t)p * n_nodes + r];
    s = warp_sum(s);
    if (lane == 0) ent[r] = s / (float)B;
}

// B operand of the output GEMM: w2t [O][Kp] bf16 with w2t[o][j l + u] = W2[j][o][u], w2t[o][2^d l + j] = b2[j][o],
// zero up to Kp.
template <typename T>
__global__ void k_pack_w2_transposed(const T* __restrict__ w2, const T* __restrict__ b2, __nv_bfloat16* __restrict__ w2t,
                                     int n_leaves, int l, int O, int Kp)
{
    const int64_t total = (int64_t)O * Kp;
    const int hidden = n_leaves * l;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t o = i / Kp;
        const int q = (int)(i % Kp);
        float v = 0.0f;
        if (q < hidden) v = Elem<T>::to_float(w2[((int64_t)(q / l) * O + o) * l + q % l]);
        else if (q < hidden + n_leaves && b2) v = Elem<T>::to_float(b2[(int64_t)(q - hidden) * O + o]);
        w2t[i] = __float2bfloat16_rn(v);
    }
}

}  // namespace fff
