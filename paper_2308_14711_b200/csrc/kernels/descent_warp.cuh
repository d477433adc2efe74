// Tree descent on CUDA cores: one warp walks one token down the tree.
//
// Algorithm 1, FORWARD_I, non-leaf branch: at node N_{m,n} the token goes to
// N_{m+1,2n+1} when sigmoid(<w,x>+b) >= 1/2, i.e. when the logit is >= 0, and
// to N_{m+1,2n} otherwise.  Each level needs the weight row selected by the
// previous decision, so the d dot products of a token are serial; the warp
// splits each of them over its lanes with 16-byte loads.
//
// This is the general path: any D, any depth, both element types.  It is the
// path of choice when few tokens share a node (deep levels, small batches),
// where every weight row is used by about one token and nothing can be reused.
#pragma once

#include "common.cuh"

namespace fff {

constexpr int kDescentWarps = 8;

// level0 / pos_in: the walk starts at node N_{level0, pos_in[t]} (pos_in NULL = position 0)
// and continues for `levels` levels; pos_out[t] receives the position reached at level
// level0 + levels.
template <typename T>
__global__ void __launch_bounds__(kDescentWarps * 32)
k_descent_warp(const T* __restrict__ x, const T* __restrict__ node_w, const T* __restrict__ node_b,
               int D, int level0, int levels, const int32_t* __restrict__ pos_in,
               int32_t* __restrict__ pos_out, int64_t B, bool vec)
{
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * kDescentWarps + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * kDescentWarps;
    for (int64_t t = warp0; t < B; t += nwarps) {
        const T* xt = x + t * D;
        int64_t n = pos_in ? pos_in[t] : 0;
        for (int m = level0; m < level0 + levels; ++m) {
            const int64_t row = ((int64_t)1 << m) - 1 + n;
            const float logit = warp_dot<T>(node_w + row * D, xt, D, vec, lane) + Elem<T>::to_float(node_b[row]);
            n = 2 * n + (logit >= 0.0f ? 1 : 0);
        }
        if (lane == 0) pos_out[t] = (int32_t)n;
    }
}

}  // namespace fff
