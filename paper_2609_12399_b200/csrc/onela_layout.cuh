// Device helpers shared by the kernel files: bf16 unpacking.
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
    static __device__ __forceinline__ void load(const float* p, float* out) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(p));
        out[0] = x.x; out[1] = x.y; out[2] = x.z; out[3] = x.w;
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(p));
        unpack_bf16x2(x.x, out[0], out[1]);
        unpack_bf16x2(x.y, out[2], out[3]);
        unpack_bf16x2(x.z, out[4], out[5]);
        unpack_bf16x2(x.w, out[6], out[7]);
    }
};

}  // namespace onela
