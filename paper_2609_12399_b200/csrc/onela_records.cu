// Shared-state store and record arena kernels.
//  - append: copy one decode call's (k, v, alpha, beta) into the append-only arena (paper Section 3.3:
//    records are written once to the slots of the current step and never relocated).
//  - store_state / prefill: fill the store slot of one (request, layer) with S_0 (Section 3.2: the
//    post-prefill state is stored once per request), either from a caller tensor or by running Eq. 1
//    from the zero state over the prompt.
#include <cuda_fp16.h>

#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {

namespace {

// One warp per (beam, head) row of one request (blockIdx.y).  The arena is head-major ([head][slot][k | v])
// so that the records one decode tile reads - consecutive beams of one head - are contiguous.
__global__ void __launch_bounds__(256) append_kernel(const char* __restrict__ k, const char* __restrict__ v,
                                                     const float* __restrict__ alpha, const float* __restrict__ beta,
                                                     char* __restrict__ kv_plane, float2* __restrict__ gate_plane,
                                                     long long arena_slots, int32_t W, int32_t H, int32_t k_bytes,
                                                     int32_t v_bytes, BatchBases bases) {
    const int r = blockIdx.y;
    const int row_in_req = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // b * H + h
    const int lane = threadIdx.x & 31;
    if (row_in_req >= W * H) return;
    const int b = row_in_req / H, h = row_in_req - b * H;
    const long long row = (long long)r * (W * H) + row_in_req;
    const long long dst_row = (long long)h * arena_slots + (bases.base[r] + b);
    const uint4* ksrc = reinterpret_cast<const uint4*>(k + row * k_bytes);
    const uint4* vsrc = reinterpret_cast<const uint4*>(v + row * v_bytes);
    uint4* dst = reinterpret_cast<uint4*>(kv_plane + dst_row * (k_bytes + v_bytes));
    const int nk = k_bytes >> 4, nv = v_bytes >> 4;
    for (int c = lane; c < nk + nv; c += 32) dst[c] = (c < nk) ? __ldg(ksrc + c) : __ldg(vsrc + (c - nk));
    if (lane == 0) gate_plane[dst_row] = make_float2(__ldg(alpha + row), __ldg(beta + row));
}

template <typename T>
__device__ __forceinline__ float to_float(T x);
template <>
__device__ __forceinline__ float to_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// The operand scale of a head (Layout::s0_scale) from the largest magnitude of its state.
__device__ __forceinline__ float operand_scale(float peak) {
    const int eb = (int)(__float_as_uint(peak) >> 23) & 255;          // biased exponent of a non-negative number
    constexpr int target = 11;                                         // scaled peak in [2^11, 2^12)
    const bool ok = eb > target + 1 && eb < 255;
    return ok ? __uint_as_float((uint32_t)(254 + target - eb) << 23) : 1.f;
}
// Largest value over the CTA (<= 1024 threads), returned to thread 0.
__device__ __forceinline__ float block_max(float v) {
    __shared__ float part[32];
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        v = threadIdx.x < (blockDim.x + 31) / 32 ? part[threadIdx.x] : 0.f;
        for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    }
    return v;
}

// Copy of the caller's states into the store, one CTA per head, with the head's operand scale as a by-product.
__global__ void __launch_bounds__(256) store_state_kernel(const float4* __restrict__ in, float4* __restrict__ out,
                                                          float* __restrict__ scale_out, int32_t vec_per_head) {
    const long long base = (long long)blockIdx.x * vec_per_head;
    float peak = 0.f;
    for (int i = threadIdx.x; i < vec_per_head; i += blockDim.x) {
        const float4 x = __ldg(in + base + i);
        out[base + i] = x;
        peak = fmaxf(fmaxf(peak, fmaxf(fabsf(x.x), fabsf(x.y))), fmaxf(fabsf(x.z), fabsf(x.w)));
    }
    peak = block_max(peak);
    if (threadIdx.x == 0) scale_out[blockIdx.x] = operand_scale(peak);
}

// Eq. 1 from the zero state over the prompt, one CTA per head, thread i owns row i of S in registers.
template <int DK, int DV, typename T>
__global__ void __launch_bounds__(DV) prefill_kernel(const T* __restrict__ k, const T* __restrict__ v,
                                                     const float* __restrict__ alpha, const float* __restrict__ beta,
                                                     float* __restrict__ slot, float* __restrict__ scale_out,
                                                     int32_t n_tokens, int32_t H) {
    __shared__ __align__(16) float k_s[2][DK];
    const int h = blockIdx.x, i = threadIdx.x;
    float S[DK];
#pragma unroll
    for (int j = 0; j < DK; ++j) S[j] = 0.f;
    constexpr int KPT = (DK + DV - 1) / DV;  // k elements each thread stages per token
    float kn[KPT], vn = 0.f, an = 1.f, bn = 0.f;
    auto fetch = [&](int t) {
        const long long row = (long long)t * H + h;
#pragma unroll
        for (int c = 0; c < KPT; ++c) {
            const int j = i + c * DV;
            kn[c] = (j < DK) ? to_float(k[row * DK + j]) : 0.f;
        }
        vn = to_float(v[row * DV + i]);
        an = __ldg(alpha + row);
        bn = __ldg(beta + row);
    };
    auto stage = [&](int buf) {
#pragma unroll
        for (int c = 0; c < KPT; ++c) {
            const int j = i + c * DV;
            if (j < DK) k_s[buf][j] = kn[c];
        }
    };
    if (n_tokens > 0) { fetch(0); stage(0); }
    __syncthreads();
    for (int t = 0; t < n_tokens; ++t) {
        const float vt = vn, a = an, b = bn;
        if (t + 1 < n_tokens) fetch(t + 1);
        const float4* kk = reinterpret_cast<const float4*>(k_s[t & 1]);
        float u0 = 0.f, u1 = 0.f, u2 = 0.f, u3 = 0.f;
#pragma unroll
        for (int j = 0; j < DK / 4; ++j) {
            const float4 x = kk[j];
            u0 = fmaf(S[4 * j + 0], x.x, u0);
            u1 = fmaf(S[4 * j + 1], x.y, u1);
            u2 = fmaf(S[4 * j + 2], x.z, u2);
            u3 = fmaf(S[4 * j + 3], x.w, u3);
        }
        const float u = (u0 + u1) + (u2 + u3);
        const float delta = b * (vt - a * u);   // Eq. 2's delta_t
#pragma unroll
        for (int j = 0; j < DK / 4; ++j) {
            const float4 x = kk[j];
            S[4 * j + 0] = fmaf(a, S[4 * j + 0], delta * x.x);
            S[4 * j + 1] = fmaf(a, S[4 * j + 1], delta * x.y);
            S[4 * j + 2] = fmaf(a, S[4 * j + 2], delta * x.z);
            S[4 * j + 3] = fmaf(a, S[4 * j + 3], delta * x.w);
        }
        if (t + 1 < n_tokens) stage((t + 1) & 1);
        __syncthreads();
    }
    float* dst = slot + (long long)h * DV * DK;
    float peak = 0.f;
#pragma unroll
    for (int j = 0; j < DK; ++j) {
        dst[(long long)i * DK + j] = S[j];
        peak = fmaxf(peak, fabsf(S[j]));
    }
    peak = block_max(peak);
    if (i == 0) scale_out[h] = operand_scale(peak);
}

template <int DK, int DV>
cudaError_t prefill_dispatch(const void* k, const void* v, const float* alpha, const float* beta, float* slot,
                             float* scale_out, int32_t n_tokens, int32_t H, int32_t rec_dtype, cudaStream_t stream) {
    if (rec_dtype == ONELA_DTYPE_BF16)
        prefill_kernel<DK, DV, __nv_bfloat16><<<H, DV, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), alpha, beta, slot, scale_out, n_tokens, H);
    else
        prefill_kernel<DK, DV, float><<<H, DV, 0, stream>>>(static_cast<const float*>(k), static_cast<const float*>(v),
                                                           alpha, beta, slot, scale_out, n_tokens, H);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_append(const void* k, const void* v, const float* alpha, const float* beta, char* kv_plane,
                          float2* gate_plane, long long arena_slots, int32_t req_count, int32_t W, int32_t H,
                          int32_t dk, int32_t dv, int32_t elem_bytes, const BatchBases& bases,
                          cudaStream_t stream) {
    const int warps_per_block = 8;
    dim3 grid((unsigned)((W * H + warps_per_block - 1) / warps_per_block), (unsigned)req_count);
    append_kernel<<<grid, warps_per_block * 32, 0, stream>>>(static_cast<const char*>(k), static_cast<const char*>(v),
                                                             alpha, beta, kv_plane, gate_plane, arena_slots, W, H,
                                                             dk * elem_bytes, dv * elem_bytes, bases);
    return cudaGetLastError();
}

// One CTA per head: the stored state as the tiled tensor-core kernel's A operand (see Layout::s0_f16).  The rounding
// is the one that kernel would do itself (x * scale to the nearest fp16), so results do not depend on who converts.
__global__ void __launch_bounds__(256) pack_state_f16_kernel(const float* __restrict__ slot, const float* __restrict__ scale,
                                                             uint16_t* __restrict__ dst, int32_t dk, int32_t dv) {
    const long long head = blockIdx.x;
    const float* S = slot + head * (long long)dv * dk;
    const float sc = scale[head];
    const int cpr = dk / 8, kb_n = dk / 64, rows = (dv + 127) / 128 * 128;     // 16-byte chunks per row, column tiles, padded rows
    char* out = reinterpret_cast<char*>(dst) + head * (long long)rows * dk * 2;
    for (int item = threadIdx.x; item < rows * cpr; item += blockDim.x) {
        const int i = item / cpr, ch = item - i * cpr;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (i < dv) {
            const float4* p = reinterpret_cast<const float4*>(S + (long long)i * dk + ch * 8);
            const float4 x0 = __ldg(p), x1 = __ldg(p + 1);
            const __half2 h0 = __floats2half2_rn(x0.x * sc, x0.y * sc), h1 = __floats2half2_rn(x0.z * sc, x0.w * sc);
            const __half2 h2 = __floats2half2_rn(x1.x * sc, x1.y * sc), h3 = __floats2half2_rn(x1.z * sc, x1.w * sc);
            w = make_uint4(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1),
                           *reinterpret_cast<const uint32_t*>(&h2), *reinterpret_cast<const uint32_t*>(&h3));
        }
        const int mt = i >> 7, row = i & 127, kb = ch >> 3, c8 = ch & 7;
        *reinterpret_cast<uint4*>(out + ((long long)(mt * kb_n + kb) * 128 + row) * 128 + ((c8 ^ (row & 7)) << 4)) = w;
    }
}

cudaError_t launch_pack_state(const float* slot, const float* scale, uint16_t* dst, long long n_heads, int32_t dk, int32_t dv,
                              cudaStream_t stream) {
    pack_state_f16_kernel<<<(unsigned)n_heads, 256, 0, stream>>>(slot, scale, dst, dk, dv);
    return cudaGetLastError();
}

cudaError_t launch_store_state(const float* S0_in, float* slot, float* scale_out, long long n_heads, int32_t dk, int32_t dv,
                               cudaStream_t stream) {
    if (n_heads <= 0 || n_heads > 0x7fffffffLL) return cudaErrorInvalidValue;
    store_state_kernel<<<(unsigned)n_heads, 256, 0, stream>>>(reinterpret_cast<const float4*>(S0_in), reinterpret_cast<float4*>(slot),
                                                             scale_out, dk * dv / 4);
    return cudaGetLastError();
}

cudaError_t launch_export_state(const float* slot, float* S0_out, int32_t H, int32_t dk, int32_t dv, cudaStream_t stream) {
    return cudaMemcpyAsync(S0_out, slot, (size_t)H * dk * dv * sizeof(float), cudaMemcpyDeviceToDevice, stream);
}

cudaError_t launch_prefill(const void* k, const void* v, const float* alpha, const float* beta, float* slot,
                           float* scale_out, int32_t n_tokens, int32_t H, int32_t dk, int32_t dv, int32_t rec_dtype,
                           bool* supported, cudaStream_t stream) {
    *supported = true;
    if (dk == 32 && dv == 32) return prefill_dispatch<32, 32>(k, v, alpha, beta, slot, scale_out, n_tokens, H, rec_dtype, stream);
    if (dk == 64 && dv == 64) return prefill_dispatch<64, 64>(k, v, alpha, beta, slot, scale_out, n_tokens, H, rec_dtype, stream);
    if (dk == 128 && dv == 128) return prefill_dispatch<128, 128>(k, v, alpha, beta, slot, scale_out, n_tokens, H, rec_dtype, stream);
    *supported = false;
    return cudaErrorInvalidValue;
}

}  // namespace onela
