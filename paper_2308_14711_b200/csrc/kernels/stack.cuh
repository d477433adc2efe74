// Glue between the FFF layers of a stack (Section "Fast feedforward layers as building blocks": an FFF layer in
// place of each feedforward layer of a transformer, i.e. behind a layer normalisation and inside a residual
// connection).  Per token, for block k:
//     x_k   = x_{k-1} + y_{k-1}                      (residual of the previous block; skipped for k = 0)
//     z_k   = (x_k - mean) / sqrt(var + eps) * gamma + beta         (mean, population variance over the D features)
// and z_k is what the block's FFF layer reads.  Both are stored in the stack's element type; the statistics are
// taken in float32 from the stored x_k (two passes: mean, then squared deviations).
// One warp per token; the row is re-read from L1/L2 between the passes (a lane re-reads only what it wrote).
// These are plain element-wise passes bound by HBM bandwidth: 2-3 reads and 1-2 writes of a [B, D] matrix.
#pragma once

#include "common.cuh"

namespace fff {

constexpr int kStackWarps = 8;

// x_out (optional, needs y_prev) = x_prev + y_prev;  z (optional) = LayerNorm(x_out or x_prev).
template <typename T>
__global__ void __launch_bounds__(kStackWarps * 32)
k_stack_glue(const T* __restrict__ x_prev, const T* __restrict__ y_prev, T* x_out, T* __restrict__ z,
             const T* __restrict__ gamma, const T* __restrict__ beta, float eps, int D, int64_t B, bool vec)
{
    pdl_trigger();
    pdl_wait();
    constexpr int V = Elem<T>::kVec;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * kStackWarps + (threadIdx.x >> 5), nwarps = (int64_t)gridDim.x * kStackWarps;
    for (int64_t t = warp0; t < B; t += nwarps) {
        const T* xp = x_prev + t * D;
        const T* cur = xp;
        float sum = 0.0f;
        if (y_prev) {
            const T* yp = y_prev + t * D;
            T* xo = x_out + t * D;
            if (vec) {
                for (int k = lane * V; k < D; k += 32 * V) {
                    float a[V], b[V];
                    Elem<T>::load_vec(xp + k, a);
                    Elem<T>::load_vec(yp + k, b);
                    __align__(16) T r[V];
#pragma unroll
                    for (int e = 0; e < V; ++e) {
                        r[e] = Elem<T>::from_float(a[e] + b[e]);
                        sum += Elem<T>::to_float(r[e]);
                    }
                    *reinterpret_cast<uint4*>(xo + k) = *reinterpret_cast<const uint4*>(r);
                }
            } else {
                for (int k = lane; k < D; k += 32) {
                    const T r = Elem<T>::from_float(Elem<T>::to_float(xp[k]) + Elem<T>::to_float(yp[k]));
                    xo[k] = r;
                    sum += Elem<T>::to_float(r);
                }
            }
            cur = xo;
        } else if (z) {
            if (vec) {
                for (int k = lane * V; k < D; k += 32 * V) {
                    float a[V];
                    Elem<T>::load_vec(xp + k, a);
#pragma unroll
                    for (int e = 0; e < V; ++e) sum += a[e];
                }
            } else {
                for (int k = lane; k < D; k += 32) sum += Elem<T>::to_float(xp[k]);
            }
        }
        if (!z) continue;
        __syncwarp();          // the row just written is read back below, in scalar mode by other lanes than wrote it
        const float mean = warp_sum(sum) / (float)D;
        // (plain loads: `cur` may be the row this warp has just written)
        float sq = 0.0f;
        if (vec) {
            for (int k = lane * V; k < D; k += 32 * V) {
                const uint4 raw = *reinterpret_cast<const uint4*>(cur + k);
                const T* r = reinterpret_cast<const T*>(&raw);
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    const float d = Elem<T>::to_float(r[e]) - mean;
                    sq = fmaf(d, d, sq);
                }
            }
        } else {
            for (int k = lane; k < D; k += 32) {
                const float d = Elem<T>::to_float(cur[k]) - mean;
                sq = fmaf(d, d, sq);
            }
        }
        const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)D + eps);
        T* zo = z + t * D;
        if (vec) {
            for (int k = lane * V; k < D; k += 32 * V) {
                const uint4 raw = *reinterpret_cast<const uint4*>(cur + k);
                const T* r = reinterpret_cast<const T*>(&raw);
                __align__(16) T out[V];
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    float v = (Elem<T>::to_float(r[e]) - mean) * rstd;
                    if (gamma) v *= Elem<T>::to_float(gamma[k + e]);
                    if (beta) v += Elem<T>::to_float(beta[k + e]);
                    out[e] = Elem<T>::from_float(v);
                }
                *reinterpret_cast<uint4*>(zo + k) = *reinterpret_cast<const uint4*>(out);
            }
        } else {
            for (int k = lane; k < D; k += 32) {
                float v = (Elem<T>::to_float(cur[k]) - mean) * rstd;
                if (gamma) v *= Elem<T>::to_float(gamma[k]);
                if (beta) v += Elem<T>::to_float(beta[k]);
                zo[k] = Elem<T>::from_float(v);
            }
        }
    }
}

}  // namespace fff
