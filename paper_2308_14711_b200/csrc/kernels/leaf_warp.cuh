// Grouped leaf evaluation on CUDA cores with un-permuting write-back.
//
// Algorithm 1, FORWARD_I, leaf branch: the token returns N_{d,j}(x), the
// <D, l, O> feedforward network of its leaf:  y = W2_j act(W1_j x + b1_j) + b2_j.
//
// One warp evaluates one token.  Warps walk the tokens in bucket order
// (perm), so the warps of a CTA mostly work on the same leaf and share its
// weights through L1/L2.  The row of y is written straight to the token's
// original position, which is the un-permute step.
//
// The kernel can also finish the descent first (tail_levels > 0): the warp walks the last levels of the tree
// from the position the staged descent reached, exactly as k_descent_warp would (same dot product, same
// comparison), records the leaf index and goes on with that leaf.  With a token per warp and no bucketing in
// between, this saves a kernel and one pass over x.
//
// General path: any D, l, O, both element types, float32 accumulation.  It is
// the path for float32 layers, for very thin leaves and for buckets of a few
// tokens, where the work is a gather of weights rather than a contraction.
#pragma once

#include "common.cuh"

namespace fff {

constexpr int kLeafWarps = 8;
constexpr int kLeafHiddenUnroll = 4;

// Dynamic shared memory: kLeafWarps * l floats (hidden activations per warp).
// kTail: walk tail_levels levels of the descent first (a separate instantiation keeps the plain kernel lean).
template <typename T, bool kTail>
__global__ void __launch_bounds__(kLeafWarps * 32)
k_leaf_warp(const T* __restrict__ x, const int32_t* __restrict__ leaf_idx, const int32_t* __restrict__ perm,
            const T* __restrict__ w1, const T* __restrict__ b1, const T* __restrict__ w2, const T* __restrict__ b2,
            T* __restrict__ y, int D, int O, int l, int act, int64_t B, bool vec,
            const T* __restrict__ node_w, const T* __restrict__ node_b, int tail_level0, int tail_levels,
            const int32_t* __restrict__ tail_pos, int32_t* __restrict__ leaf_out)
{
    extern __shared__ float s_h[];
    pdl_trigger();
    pdl_wait();
    constexpr int V = Elem<T>::kVec;
    constexpr int U = kLeafHiddenUnroll;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    float* h = s_h + (size_t)wib * l;
    const int64_t warp0 = (int64_t)blockIdx.x * kLeafWarps + wib;
    const int64_t nwarps = (int64_t)gridDim.x * kLeafWarps;

    for (int64_t i = warp0; i < B; i += nwarps) {
        const int64_t t = perm ? perm[i] : i;
        const T* xt = x + t * D;
        int64_t j;
        if (kTail) {
            // the walk starts at node N_{tail_level0, tail_pos[t]} (position 0 without tail_pos)
            int64_t n = tail_pos ? tail_pos[t] : 0;
            for (int m = tail_level0; m < tail_level0 + tail_levels; ++m) {
                const int64_t row = ((int64_t)1 << m) - 1 + n;
                const float logit = warp_dot<T>(node_w + row * D, xt, D, vec, lane) + Elem<T>::to_float(node_b[row]);
                n = 2 * n + (logit >= 0.0f ? 1 : 0);
            }
            j = n;
            if (lane == 0) leaf_out[t] = (int32_t)n;
        } else {
            j = leaf_idx[t];
        }
        const T* w1j = w1 + j * (int64_t)l * D;
        const T* b1j = b1 + j * (int64_t)l;

        // hidden layer: U neurons at a time share the loads of x
        for (int i0 = 0; i0 < l; i0 += U) {
            float acc[U];
#pragma unroll
            for (int u = 0; u < U; ++u) acc[u] = 0.0f;
            if (vec) {
                for (int k = lane * V; k < D; k += 32 * V) {
                    float fx[V];
                    Elem<T>::load_vec(xt + k, fx);
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (i0 + u < l) {
                            float fw[V];
                            Elem<T>::load_vec(w1j + (int64_t)(i0 + u) * D + k, fw);
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[u] = fmaf(fw[e], fx[e], acc[u]);
                        }
                    }
                }
            } else {
                for (int k = lane; k < D; k += 32) {
                    const float fx = Elem<T>::to_float(xt[k]);
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (i0 + u < l) acc[u] = fmaf(Elem<T>::to_float(w1j[(int64_t)(i0 + u) * D + k]), fx, acc[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float s = warp_sum(acc[u]);
                if (lane == 0 && i0 + u < l) h[i0 + u] = activate(act, s + Elem<T>::to_float(b1j[i0 + u]));
            }
        }
        __syncwarp();

        // output layer.  Thin leaves (l = 1, rows of W2 are single elements): 8 / 4 consecutive outputs per
        // lane with 16-byte loads of W2, b2 and a 16-byte store of y.  Otherwise one output neuron per lane,
        // four rows in flight.
        const T* w2j = w2 + j * (int64_t)O * l;
        const T* b2j = b2 + j * (int64_t)O;
        T* yt = y + t * O;
        if (l == 1 && vec && (O % V) == 0) {
            const float h0 = h[0];
            for (int o = lane * V; o < O; o += 32 * V) {
                float fw[V], fb[V];
                Elem<T>::load_vec(w2j + o, fw);
                Elem<T>::load_vec(b2j + o, fb);
                alignas(16) T out[V];
#pragma unroll
                for (int e = 0; e < V; ++e) out[e] = Elem<T>::from_float(fmaf(fw[e], h0, fb[e]));
                *reinterpret_cast<uint4*>(yt + o) = *reinterpret_cast<const uint4*>(out);
            }
        } else {
#pragma unroll 4
            for (int o = lane; o < O; o += 32) {
                const T* row = w2j + (int64_t)o * l;
                float acc = Elem<T>::to_float(b2j[o]);
                for (int q = 0; q < l; ++q) acc = fmaf(Elem<T>::to_float(row[q]), h[q], acc);
                yt[o] = Elem<T>::from_float(acc);
            }
        }
        __syncwarp();
    }
}

}  // namespace fff
