// Whole forward pass in one launch for small trees with thin leaves (the regime of the paper's own
// timing tables: a few hundred inputs, leaves of at most 32 neurons, a few thousand tokens).
//
// Algorithm 1, FORWARD_I, both branches.  The three-kernel path (descent, bucketing, grouped leaf
// evaluation) is bound by launch latency here: the whole problem is a few megabytes.  This kernel is
// organised by LEAF, not by token: the hidden neurons of the tree are cut into groups of 32 (one leaf of
// width 32, or 32 / lp leaves of padded width lp), and CTA (g, s) keeps the hidden-layer weights of
// group g in shared memory for its whole life and serves the tokens of token slice s that were routed
// into a leaf of group g.  No bucketing and no permutation exist at all: a CTA finds its tokens by
// scanning the leaf indices of its slice.
//
//   phase A   the CTAs share the tokens evenly; one warp walks one token down the tree (the same dot
//             product and comparison as k_descent_warp) and records its leaf.  Meanwhile the bulk
//             copy of the CTA's weight group is in flight.
//   barrier   one grid-wide barrier (the launch is cooperative, so all CTAs are resident).
//   phase B   per batch of up to 32 of its tokens: the token rows go to shared memory (transposed); the
//             16 warps split the input dimension, every lane keeps a 4-neuron x 2/4/8-token block of
//             partial sums in registers (fused_hidden_pass); the partial sums are added across warps in
//             a fixed order, bias and activation follow, and the output layer (l products per output,
//             only the neurons of the token's own leaf) writes y at the token's own position.
//
// float32 accumulation throughout; every token's result is independent of which tokens share its
// batch, so outputs are bit-reproducible.
//
// Requirements: l <= 32, at most gridDim.x / S groups, cooperative launch, shared memory for one group
// of hidden weights, the group's output weights and one token batch.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"
#include "ptx.cuh"

namespace fff {

constexpr int kFSWarps = 16;
constexpr int kFSThreads = kFSWarps * 32;
constexpr int kFSMaxBatch = 32;           // tokens evaluated together in phase B (a handle may use 16 or 8: shared memory)
constexpr int kFSListCap = kFSThreads;    // tokens of a slice examined per round: one per thread
constexpr int kFSRowRegs = 8;             // 16-byte vectors of a token row that a lane keeps in registers during the descent

// Hidden-layer image of the fused kernel: [group][Dp inputs][32 neurons] float32, Dp = D rounded up to 4,
// neuron (j % LPG) * lp + i of group j / LPG is unit i of leaf j; absent neurons and columns are zero.
// b1g: [group][32];  w2g: [group][O][32] (column = neuron of the group);  b2f: [leaf][O] float32.
template <typename T>
__global__ void k_pack_fused_small(const T* __restrict__ w1, const T* __restrict__ b1, const T* __restrict__ w2,
                                   const T* __restrict__ b2, float* __restrict__ w1g, float* __restrict__ b1g,
                                   float* __restrict__ w2g, float* __restrict__ b2f, int n_leaves, int l, int lp, int D, int Dp,
                                   int O, int G)
{
    const int LPG = 32 / lp;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t n1 = (int64_t)G * Dp * 32;
    for (int64_t i = t0; i < n1; i += stride) {
        const int n = (int)(i & 31);
        const int64_t k = (i >> 5) % Dp, g = (i >> 5) / Dp;
        const int64_t leaf = g * LPG + n / lp;
        const int u = n % lp;
        w1g[i] = (leaf < n_leaves && u < l && k < D) ? Elem<T>::to_float(w1[(leaf * l + u) * D + k]) : 0.0f;
    }
    for (int64_t i = t0; i < (int64_t)G * 32; i += stride) {
        const int n = (int)(i & 31);
        const int64_t leaf = (i >> 5) * LPG + n / lp;
        const int u = n % lp;
        b1g[i] = (leaf < n_leaves && u < l && b1) ? Elem<T>::to_float(b1[leaf * l + u]) : 0.0f;
    }
    for (int64_t i = t0; i < (int64_t)G * O * 32; i += stride) {
        const int n = (int)(i & 31);
        const int64_t o = (i >> 5) % O, g = (i >> 5) / O, leaf = g * LPG + n / lp;
        const int u = n % lp;
        w2g[i] = (leaf < n_leaves && u < l) ? Elem<T>::to_float(w2[(leaf * O + o) * l + u]) : 0.0f;
    }
    for (int64_t i = t0; i < (int64_t)n_leaves * O; i += stride) b2f[i] = b2 ? Elem<T>::to_float(b2[i]) : 0.0f;
}

// Shared-memory layout (bytes), in this order: hidden weights [Dp][32], output weights [O][32], output biases of
// the group's leaves [32 / lp][O] (at most [32][O]), the staging area (token batch [Dp][batch], transposed; later the
// partial sums [warp][batch][32]), hidden activations [batch][32], hidden bias [32], token list, barrier, warp counts.
struct FusedSmallLayout {
    int Dp, O, batch;
    __host__ __device__ size_t w1_bytes() const { return (size_t)32 * Dp * 4; }
    __host__ __device__ size_t w2_bytes() const { return (size_t)O * 32 * 4; }
    __host__ __device__ size_t b2_bytes() const { return (size_t)O * 32 * 4; }
    __host__ __device__ size_t stage_bytes() const { return (size_t)(Dp > kFSWarps * 32 ? Dp : kFSWarps * 32) * batch * 4; }
    __host__ __device__ size_t h_bytes() const { return (size_t)batch * 32 * 4; }
    __host__ __device__ size_t total() const {
        return w1_bytes() + w2_bytes() + b2_bytes() + stage_bytes() + h_bytes() + 128 + kFSListCap * 8 + 8 + kFSWarps * 4 + 56;
    }
};

// One warp's share of the hidden layer for a batch of 4 * TT tokens: lane (lt, ln) = (lane / 8, lane % 8) owns
// the neurons 4 ln .. 4 ln + 3 and the tokens TT lt .. TT lt + TT - 1 and keeps their 4 x TT partial sums in
// registers.  Per input k: one 16-byte load of four weights (the eight lanes of a quarter warp read 128
// consecutive bytes) and TT / 4 16-byte loads of tokens (one address per quarter warp) feed 4 TT multiply-adds;
// with one neuron per lane and broadcast tokens the shared-memory pipe, not the arithmetic, set the pace.
// xs: [k][4 * TT] tokens;  part: this warp's [4 * TT tokens][32 neurons] partial sums.
template <int TT>
__device__ __forceinline__ void fused_hidden_pass(const float* __restrict__ w1s, const float* __restrict__ xs, int ka, int kb,
                                                  float (&acc)[4][TT], int lane)
{
    const int ln = lane & 7, lt = lane >> 3;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TT; ++j) acc[i][j] = 0.0f;
#pragma unroll 2
    for (int k = ka; k < kb; ++k) {
        const float4 w = *reinterpret_cast<const float4*>(w1s + k * 32 + ln * 4);
        float xv[TT];
        if constexpr (TT == 2) {
            const float2 v = *reinterpret_cast<const float2*>(xs + k * (4 * TT) + lt * TT);
            xv[0] = v.x; xv[1] = v.y;
        } else {
#pragma unroll
            for (int q = 0; q < TT / 4; ++q) {
                const float4 v = *reinterpret_cast<const float4*>(xs + k * (4 * TT) + lt * TT + q * 4);
                xv[4 * q] = v.x; xv[4 * q + 1] = v.y; xv[4 * q + 2] = v.z; xv[4 * q + 3] = v.w;
            }
        }
#pragma unroll
        for (int j = 0; j < TT; ++j) {
            acc[0][j] = fmaf(w.x, xv[j], acc[0][j]);
            acc[1][j] = fmaf(w.y, xv[j], acc[1][j]);
            acc[2][j] = fmaf(w.z, xv[j], acc[2][j]);
            acc[3][j] = fmaf(w.w, xv[j], acc[3][j]);
        }
    }
}

template <int TT>
__device__ __forceinline__ void fused_store_partials(float* __restrict__ part_warp, const float (&acc)[4][TT], int lane)
{
    const int ln = lane & 7, lt = lane >> 3;
#pragma unroll
    for (int j = 0; j < TT; ++j)
        *reinterpret_cast<float4*>(part_warp + (lt * TT + j) * 32 + ln * 4) = make_float4(acc[0][j], acc[1][j], acc[2][j], acc[3][j]);
}

// grid = G * S CTAs: CTA c serves group c % G and token slice c / G.
// leaf_out: [B] leaf of every token (always written; read again after the grid barrier); leaf_out2: optional copy.
template <typename T>
__global__ void __launch_bounds__(kFSThreads, 1)
k_fused_small(const T* __restrict__ x, const T* __restrict__ node_w, const T* __restrict__ node_b,
              const float* __restrict__ w1g, const float* __restrict__ b1g, const float* __restrict__ w2g,
              const float* __restrict__ b2f, T* __restrict__ y, int32_t* leaf_out, int32_t* __restrict__ leaf_out2,
              int D, int Dp, int O, int depth, int l, int lp, int act, int B, int G, int batch, int vec, int n_leaves,
              int* __restrict__ status)
{
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) unsigned char smem_fs[];
    const FusedSmallLayout L{Dp, O, batch};
    float* w1s = reinterpret_cast<float*>(smem_fs);
    float* w2s = reinterpret_cast<float*>(smem_fs + L.w1_bytes());
    float* b2s = w2s + (size_t)O * 32;
    float* stage = b2s + (size_t)O * 32;
    float* hs = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(stage) + L.stage_bytes());
    float* b1s = hs + (size_t)batch * 32;
    int* list_tok = reinterpret_cast<int*>(b1s + 32);
    int* list_leaf = list_tok + kFSListCap;
    uint64_t* bar = reinterpret_cast<uint64_t*>(list_leaf + kFSListCap);
    int* s_wcnt = reinterpret_cast<int*>(bar + 1);           // [kFSWarps]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = blockIdx.x % G, s = blockIdx.x / G, S = gridDim.x / G;
    const int LPG = 32 / lp;

    // the weight group starts to arrive while phase A runs
    if (tid == 0) {
        ptx::mbar_init(bar, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (tid == 0) {
        const uint32_t bytes = (uint32_t)L.w1_bytes();          // 128 * Dp: a multiple of 16, below the shared-memory size
        ptx::mbar_arrive_expect_tx(bar, bytes);
        ptx::bulk_g2s(w1s, reinterpret_cast<const unsigned char*>(w1g) + (size_t)g * bytes, bytes, bar);
    }
    for (int i = tid; i < O * 32; i += kFSThreads) w2s[i] = w2g[(size_t)g * O * 32 + i];
    for (int i = tid; i < LPG * O; i += kFSThreads) {
        const int64_t leaf = (int64_t)g * LPG + i / O;
        b2s[i] = leaf < n_leaves ? b2f[leaf * O + i % O] : 0.0f;
    }
    if (tid < 32) b1s[tid] = b1g[g * 32 + tid];

    // ---- phase A: descent, tokens shared evenly by all CTAs, one warp per token.  The token row stays in
    // registers for all levels (rows of up to kFSRowRegs * 32 vectors), all loads of a level are issued at once.
    {
        constexpr int V = Elem<T>::kVec;
        const int per = (B + (int)gridDim.x - 1) / (int)gridDim.x;
        const int a0 = min((int)blockIdx.x * per, B), a1 = min(a0 + per, B);
        const bool in_regs = vec != 0 && D <= kFSRowRegs * 32 * V;
        for (int t = a0 + warp; t < a1; t += kFSWarps) {
            const T* xt = x + (int64_t)t * D;
            int64_t n = 0;
            if (in_regs) {
                float xr[kFSRowRegs][V];
#pragma unroll
                for (int i = 0; i < kFSRowRegs; ++i) {
                    const int k = (i * 32 + lane) * V;
                    if (k < D) {
                        Elem<T>::load_vec(xt + k, xr[i]);
                    } else {
#pragma unroll
                        for (int e = 0; e < V; ++e) xr[i][e] = 0.0f;
                    }
                }
                for (int m = 0; m < depth; ++m) {
                    const int64_t row = ((int64_t)1 << m) - 1 + n;
                    const T* wr = node_w + row * D;
                    float fw[kFSRowRegs][V];
#pragma unroll
                    for (int i = 0; i < kFSRowRegs; ++i) {
                        const int k = (i * 32 + lane) * V;
                        if (k < D) {
                            Elem<T>::load_vec(wr + k, fw[i]);
                        } else {
#pragma unroll
                            for (int e = 0; e < V; ++e) fw[i][e] = 0.0f;
                        }
                    }
                    float acc = 0.0f;
#pragma unroll
                    for (int i = 0; i < kFSRowRegs; ++i)
#pragma unroll
                        for (int e = 0; e < V; ++e) acc = fmaf(fw[i][e], xr[i][e], acc);
                    const float logit = warp_sum(acc) + Elem<T>::to_float(node_b[row]);
                    n = 2 * n + (logit >= 0.0f ? 1 : 0);
                }
            } else {
                for (int m = 0; m < depth; ++m) {
                    const int64_t row = ((int64_t)1 << m) - 1 + n;
                    const float logit = warp_dot<T>(node_w + row * D, xt, D, vec != 0, lane) + Elem<T>::to_float(node_b[row]);
                    n = 2 * n + (logit >= 0.0f ? 1 : 0);
                }
            }
            if (lane == 0) {
                leaf_out[t] = (int32_t)n;
                if (leaf_out2) leaf_out2[t] = (int32_t)n;
            }
        }
    }
    __threadfence();
    cg::this_grid().sync();

    // ---- phase B: the tokens of slice s that were routed into group g
    bool timed_out = false;
    if (!ptx::mbar_wait(bar, 0)) timed_out = true;        // the weight group has landed
    const int TS = (B + S - 1) / S;
    const int s0 = min(s * TS, B), s1 = min(s0 + TS, B);
    const int kper = (Dp + kFSWarps - 1) / kFSWarps;
    const int ka = min(warp * kper, Dp), kb = min(ka + kper, Dp);

    for (int r0 = s0; r0 < s1; r0 += kFSListCap) {
        // tokens of this round that belong to the group, in token order (ballot ranks inside a warp, then the
        // counts of the warps before); one token per thread
        __syncthreads();
        const int t_mine = r0 + tid;
        int leaf_mine = -1;
        if (t_mine < s1) leaf_mine = __ldcg(leaf_out + t_mine);
        const bool in = leaf_mine >= 0 && leaf_mine / LPG == g;
        const unsigned m = __ballot_sync(kFullMask, in);
        if (lane == 0) s_wcnt[warp] = __popc(m);
        __syncthreads();
        int before = 0, n_list = 0;
        for (int w = 0; w < kFSWarps; ++w) {
            const int c = s_wcnt[w];
            if (w < warp) before += c;
            n_list += c;
        }
        if (in) {
            const int pos = before + __popc(m & ((1u << lane) - 1u));
            list_tok[pos] = t_mine;
            list_leaf[pos] = leaf_mine;
        }
        __syncthreads();

        for (int c0 = 0; c0 < n_list; c0 += batch) {
            const int tb = min(batch, n_list - c0);
            const int TT = tb <= 8 ? 2 : tb <= 16 ? 4 : 8;       // tokens per lane; the staged rows hold 4 TT tokens
            const int RS = 4 * TT;
            // token rows -> shared memory as float32, transposed: stage[k][token]; tokens past tb and inputs past D
            // are zero.  A thread moves 32 bytes of one row at a time; consecutive threads take consecutive tokens.
            __syncthreads();
            if (vec) {
                constexpr int V = Elem<T>::kVec, R = 32 / (int)sizeof(T) / V;      // vectors per 32 bytes
                constexpr int U = 4;                                               // pieces in flight per thread
                const int chunks = (D + V * R - 1) / (V * R);
                for (int i0 = tid; i0 < RS * chunks; i0 += U * kFSThreads) {
                    float f[U][R][V];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int i = i0 + u * kFSThreads;
                        const int t = i % RS, k0 = (i / RS) * (V * R);
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            if (i < RS * chunks && t < tb && k0 + r * V < D) {
                                Elem<T>::load_vec(x + (int64_t)list_tok[c0 + t] * D + k0 + r * V, f[u][r]);
                            } else {
#pragma unroll
                                for (int e = 0; e < V; ++e) f[u][r][e] = 0.0f;
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int i = i0 + u * kFSThreads;
                        const int t = i % RS, k0 = (i / RS) * (V * R);
                        if (i < RS * chunks) {
#pragma unroll
                            for (int r = 0; r < R; ++r)
#pragma unroll
                                for (int e = 0; e < V; ++e)
                                    if (k0 + r * V + e < Dp) stage[(size_t)(k0 + r * V + e) * RS + t] = f[u][r][e];
                        }
                    }
                }
            } else {
                for (int i = tid; i < RS * Dp; i += kFSThreads) {
                    const int t = i % RS, k = i / RS;
                    stage[i] = (t < tb && k < D) ? Elem<T>::to_float(x[(int64_t)list_tok[c0 + t] * D + k]) : 0.0f;
                }
            }
            __syncthreads();

            // hidden layer: this warp's share of the input dimension; then the partial sums take the place of the tokens
            float* part_warp = stage + (size_t)warp * RS * 32;
            if (TT == 2) {
                float acc[4][2];
                fused_hidden_pass<2>(w1s, stage, ka, kb, acc, lane);
                __syncthreads();
                fused_store_partials<2>(part_warp, acc, lane);
            } else if (TT == 4) {
                float acc[4][4];
                fused_hidden_pass<4>(w1s, stage, ka, kb, acc, lane);
                __syncthreads();
                fused_store_partials<4>(part_warp, acc, lane);
            } else {
                float acc[4][8];
                fused_hidden_pass<8>(w1s, stage, ka, kb, acc, lane);
                __syncthreads();
                fused_store_partials<8>(part_warp, acc, lane);
            }
            __syncthreads();
            // sum over the warps in warp order, bias, activation
            for (int i = tid; i < tb * 32; i += kFSThreads) {
                const int t = i >> 5, n = i & 31;
                float sum = b1s[n];
                for (int w = 0; w < kFSWarps; ++w) sum += stage[((size_t)w * RS + t) * 32 + n];
                hs[i] = activate(act, sum);
            }
            __syncthreads();
            // output layer: only the neurons of the token's own leaf
            for (int i = tid; i < tb * O; i += kFSThreads) {
                const int t = i / O, o = i % O;
                const int lq = list_leaf[c0 + t] % LPG, n0 = lq * lp;
                // (four running sums: the shared-memory loads of one do not wait for the additions of another)
                float sum[4] = {b2s[lq * O + o], 0.0f, 0.0f, 0.0f};
                const float* wr = w2s + o * 32 + n0;
                const float* hr = hs + t * 32 + n0;
                int u = 0;
                for (; u + 4 <= l; u += 4) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) sum[q] = fmaf(wr[u + q], hr[u + q], sum[q]);
                }
                for (; u < l; ++u) sum[0] = fmaf(wr[u], hr[u], sum[0]);
                y[(int64_t)list_tok[c0 + t] * O + o] = Elem<T>::from_float((sum[0] + sum[1]) + (sum[2] + sum[3]));
            }
        }
    }
    if (timed_out && tid == 0) atomicExch(status, kDevTimeout);
}

}  // namespace fff
