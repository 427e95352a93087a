// Device helpers shared by the kernel files: bf16 unpacking and packing, vector stores of fp32 results.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace onela {

// Two packed bf16 (little endian: element 0 in the low half) -> two fp32, exactly.
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}

template <typename T>
struct Vec16;  // one 16-byte vector of T, unpacked to fp32
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4& x, float* out) {
        out[0] = __uint_as_float(x.x); out[1] = __uint_as_float(x.y); out[2] = __uint_as_float(x.z); out[3] = __uint_as_float(x.w);
    }
    static __device__ __forceinline__ void load(const float* p, float* out) { unpack(__ldg(reinterpret_cast<const uint4*>(p)), out); }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4& x, float* out) {
        unpack_bf16x2(x.x, out[0], out[1]);
        unpack_bf16x2(x.y, out[2], out[3]);
        unpack_bf16x2(x.z, out[4], out[5]);
        unpack_bf16x2(x.w, out[6], out[7]);
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) { unpack(__ldg(reinterpret_cast<const uint4*>(p)), out); }
};

// two fp32 -> two packed bf16 (element 0 in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
// VEC consecutive outputs of type OutT from fp32 (VEC = 4 or 8: the elements of one 16-byte vector of the record type)
template <typename OutT, int VEC>
__device__ __forceinline__ void store_out(OutT* p, const float* x) {
    if constexpr (sizeof(OutT) == 4) {
#pragma unroll
        for (int e = 0; e < VEC; e += 4) *reinterpret_cast<float4*>(p + e) = make_float4(x[e], x[e + 1], x[e + 2], x[e + 3]);
    } else if constexpr (VEC == 8) {
        *reinterpret_cast<uint4*>(p) = make_uint4(pack2(x[0], x[1]), pack2(x[2], x[3]), pack2(x[4], x[5]), pack2(x[6], x[7]));
    } else {
        *reinterpret_cast<uint2*>(p) = make_uint2(pack2(x[0], x[1]), pack2(x[2], x[3]));
    }
}

}  // namespace onela
