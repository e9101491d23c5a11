// How one warp covers the heads of a node row [H, D] with 16-byte loads.
//
// G consecutive lanes share one head; load j of lane `sub` (= lane % G) takes the VEC
// elements starting at (j*G + sub)*VEC, so each load instruction of the G lanes covers
// G*16 contiguous bytes and a warp covers 32/G heads (a full 1 KB row for bf16, d=64, H=8).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace bpt {

// 2^x with the hardware approximation (about 2 ulp; -inf gives 0)
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T> struct Elem;

template <> struct Elem<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void load(const float* p, float* x) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void store(float* p, const float* x) {
        *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};

template <> struct Elem<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* x) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float* x) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <typename T, int D> struct RowMap {
    static constexpr int VEC = Elem<T>::VEC;
    static constexpr int G = sizeof(T) == 4 ? 8 : 4;  // lanes per head
    static constexpr int EPL = D / G;                 // elements per lane
    static constexpr int NV = EPL / VEC;              // 16-byte loads per lane and row
    static constexpr int HPW = 32 / G;                // heads per warp
    static_assert(NV >= 1 && NV * VEC == EPL, "row does not split into 16-byte pieces");

    // `head_row` points at the D elements of one head.
    static __device__ __forceinline__ void load(const T* head_row, int sub, float* x) {
#pragma unroll
        for (int j = 0; j < NV; ++j) Elem<T>::load(head_row + (j * G + sub) * VEC, x + j * VEC);
    }
    static __device__ __forceinline__ void store(T* head_row, int sub, const float* x) {
#pragma unroll
        for (int j = 0; j < NV; ++j) Elem<T>::store(head_row + (j * G + sub) * VEC, x + j * VEC);
    }
    // sum over the G lanes of a head; every lane gets the result
    static __device__ __forceinline__ float head_sum(float x) {
#pragma unroll
        for (int o = 1; o < G; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        return x;
    }
};

}  // namespace bpt
