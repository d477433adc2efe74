// Shared device helpers for the FFF inference kernels (sm_100a).
#pragma once

#include <type_traits>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fff {

constexpr unsigned kFullMask = 0xffffffffu;

enum : int { kActRelu = 0, kActGelu = 1, kActGeluTanh = 2, kActSilu = 3 };

// Values written to the per-handle device status word by kernels.
enum : int { kDevOk = 0, kDevTimeout = 1 };

// A tile of the grouped kernels: up to a fixed number of consecutive perm entries of one bin
// (a leaf, or a node position during a staged descent).
struct Tile {
    int bin, start, rows, pad;
};

// Programmatic dependent launch.  pdl_trigger: the next kernel in the stream may be scheduled from now
// on.  pdl_wait: block until the previous kernel in the stream has completed and its writes are
// visible; must precede the first read of anything that kernel produced.  Both are no-ops for a
// kernel that was launched the ordinary way.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename T> struct Elem;


template <> struct Elem<float> {
    static constexpr int kVec = 4;   // elements per 16-byte load
    __device__ __forceinline__ static float to_float(float v) { return v; }
    __device__ __forceinline__ static float from_float(float v) { return v; }
    __device__ __forceinline__ static void load_vec(const float* p, float (&out)[4]) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};

template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ __forceinline__ static float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ __forceinline__ static __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
    __device__ __forceinline__ static void load_vec(const __nv_bfloat16* p, float (&out)[8]) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);              // low half = even element
            out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);  // high half = odd element
        }
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    return v;
}

// The leaf's hidden activation (create-time parameter; the paper's Definition leaves it open): ReLU, GELU in
// the exact erf form, GELU in the published tanh form v/2 (1 + tanh(sqrt(2/pi) (v + 0.044715 v^3))), SiLU
// v sigmoid(v).  All four map 0 to 0, which the zero-padded hidden units of the tensor-core images rely on.
__device__ __forceinline__ float activate(int act, float v) {
    if (act == kActRelu) return fmaxf(v, 0.0f);
    if (act == kActGeluTanh) return 0.5f * v * (1.0f + tanhf(0.79788456080286535588f * (v + 0.044715f * v * v * v)));
    if (act == kActSilu) return v / (1.0f + expf(-v));
    return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
}

// The same for kernels whose result is rounded to bf16 right away: erf by the rational-times-exponential
// formula 7.1.26 of Abramowitz & Stegun (absolute error below 1.5e-7, far inside half a bf16 ulp of the
// GELU value), one exponential and one division instead of the long polynomial of erff.
__device__ __forceinline__ float activate_bf16(int act, float v) {
    if (act == kActRelu) return fmaxf(v, 0.0f);
    if (act == kActGeluTanh) {
        // tanh(u) = 1 - 2 / (1 + e^(2u)), u clamped where tanh is +-1 to float32 anyway (keeps e^(2u) finite)
        const float u = fminf(fmaxf(0.79788456080286535588f * (v + 0.044715f * v * v * v), -15.0f), 15.0f);
        const float th = 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * u));
        return 0.5f * v * (1.0f + th);
    }
    if (act == kActSilu) return v * __fdividef(1.0f, 1.0f + __expf(-fmaxf(v, -80.0f)));      // e^80 is finite; below, the result is -0
    const float z = fabsf(v) * 0.70710678118654752440f;
    const float t = __fdividef(1.0f, fmaf(0.3275911f, z, 1.0f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    const float e = 1.0f - poly * t * __expf(-z * z);          // erf(|v| / sqrt 2)
    return 0.5f * v * (1.0f + copysignf(e, v));
}

// Calls f(std::integral_constant<int, act>) with the activation as a compile-time constant.  Code that applies the
// activation to many values in an unrolled loop goes through this: with a run-time `act` every value carries the
// branches between the four forms, which keeps the values' dependency chains from overlapping.
template <class F>
__device__ __forceinline__ void with_activation(int act, F&& f) {
    switch (act) {
        case kActRelu: f(std::integral_constant<int, kActRelu>{}); break;
        case kActGeluTanh: f(std::integral_constant<int, kActGeluTanh>{}); break;
        case kActSilu: f(std::integral_constant<int, kActSilu>{}); break;
        default: f(std::integral_constant<int, kActGelu>{}); break;
    }
}

// <a, b> over n elements, evaluated by one warp; every lane returns the sum.
// `vec` says both rows start on 16-byte boundaries and n is a multiple of kVec.
template <typename T>
__device__ __forceinline__ float warp_dot(const T* __restrict__ a, const T* __restrict__ b, int n, bool vec, int lane) {
    constexpr int V = Elem<T>::kVec;
    float acc = 0.0f;
    if (vec) {
        for (int k = lane * V; k < n; k += 32 * V) {
            float fa[V], fb[V];
            Elem<T>::load_vec(a + k, fa);
            Elem<T>::load_vec(b + k, fb);
#pragma unroll
            for (int i = 0; i < V; ++i) acc = fmaf(fa[i], fb[i], acc);
        }
    } else {
        for (int k = lane; k < n; k += 32) acc = fmaf(Elem<T>::to_float(a[k]), Elem<T>::to_float(b[k]), acc);
    }
    return warp_sum(acc);
}

}  // namespace fff
