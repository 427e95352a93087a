// Grouped value heads: Hv value heads share Hk = Hv / g key heads (value head j reads the queries and keys of key
// head j / g; states, values, gates and outputs are per value head).  The operator suite the paper evaluates has
// such shapes (Section 4.1); the record then splits: k is stored once per KEY head, v and the gates per VALUE head,
// which is what saves record bytes.  CUDA cores; one CTA = (request, value head, tile of 32 beams); the fold and
// the contraction are those of the ungrouped CUDA-core kernel (see onela_decode_generic.cu) with the key side read
// from the key head's plane.
#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {

namespace {

constexpr int NB = 32;  // beams per tile

template <int DK, int DV, typename T, typename OutT, int G>
__global__ void __launch_bounds__(NB* G) decode_grouped_kernel(const GroupedArgs a) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int CK = DK / (G * VEC), CV = DV / (G * VEC);  // 16-byte chunks per lane
    static_assert(CK >= 1 && CV >= 1 && DK % (G * VEC) == 0 && DV % (G * VEC) == 0, "lane mapping");
    static_assert((DV / G) % 4 == 0, "row bands of the contraction");
    constexpr int RP = DK + 4, CP = DV + 4;  // padded pitches (floats): conflict-free 16-byte accesses
    extern __shared__ __align__(16) float smem[];
    float* R_s = smem;             // [NB][RP]  folded queries
    float* C_s = smem + NB * RP;   // [NB][CP]  corr, then the finished outputs

    const int tile = blockIdx.x, hv = blockIdx.y, req = blockIdx.z;
    const int hk = hv / a.g, Hv = a.Hk * a.g;
    const int grp = threadIdx.x / G, g = threadIdx.x % G;
    const int b = tile * NB + grp;
    const bool active = b < a.W;
    const int bb = active ? b : a.W - 1;  // idle groups shadow a live beam so loads and shuffles stay uniform

    const T* q = static_cast<const T*>(a.q) + (((long long)req * a.W + bb) * a.Hk + hk) * DK;
    const int32_t* table = a.table + req * a.table_req_stride;
    const T* kplane = reinterpret_cast<const T*>(a.kplane) + (long long)hk * a.arena_slots * DK;
    const T* vplane = reinterpret_cast<const T*>(a.vplane) + (long long)hv * a.arena_slots * DV;
    const float2* gates = a.gates + (long long)hv * a.arena_slots;

    float r[CK * VEC], corr[CV * VEC];
#pragma unroll
    for (int c = 0; c < CK; ++c) Vec16<T>::load(q + (c * G + g) * VEC, r + c * VEC);
#pragma unroll
    for (int e = 0; e < CV * VEC; ++e) corr[e] = 0.f;

    float decay = 1.f;  // product of the alphas already passed
    for (int level = a.depth - 1; level >= 0; --level) {
        const int32_t slot = (level == a.depth - 1) ? a.bases.base[req] + bb
                                                    : __ldg(table + (long long)level * a.max_beam + bb);
        const T* krec = kplane + (long long)slot * DK;
        const T* vrec = vplane + (long long)slot * DV;
        const float2 gate = __ldg(gates + slot);
        float kx[CK * VEC];
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            Vec16<T>::load(krec + (c * G + g) * VEC, kx + c * VEC);
#pragma unroll
            for (int e = 0; e < VEC; ++e) dot = fmaf(kx[c * VEC + e], r[c * VEC + e], dot);
        }
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        const float bc = gate.y * dot;        // beta_j * (k_j . r~_j)
        const float wv = decay * bc;
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            float vx[VEC];
            Vec16<T>::load(vrec + (c * G + g) * VEC, vx);
#pragma unroll
            for (int e = 0; e < VEC; ++e) corr[c * VEC + e] = fmaf(wv, vx[e], corr[c * VEC + e]);
        }
#pragma unroll
        for (int e = 0; e < CK * VEC; ++e) r[e] = fmaf(-bc, kx[e], r[e]);
        decay *= gate.x;
    }

#pragma unroll
    for (int c = 0; c < CK; ++c)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
            const int o = c * VEC + e;
            *reinterpret_cast<float4*>(R_s + grp * RP + (c * G + g) * VEC + e) =
                make_float4(decay * r[o], decay * r[o + 1], decay * r[o + 2], decay * r[o + 3]);
        }
#pragma unroll
    for (int c = 0; c < CV; ++c)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
            const int o = c * VEC + e;
            *reinterpret_cast<float4*>(C_s + grp * CP + (c * G + g) * VEC + e) =
                make_float4(corr[o], corr[o + 1], corr[o + 2], corr[o + 3]);
        }
    __syncthreads();

    // out[beam][i] = sum_k S0[i][k] R[beam][k] + corr[beam][i]; lane = beam, warp = band of DV/G rows
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const float* S0h = a.s0 + req * a.s0_req_stride + (long long)hv * DV * DK;
        const float* Rl = R_s + lane * RP;
        constexpr int ROWS = DV / G;
        for (int i0 = warp * ROWS; i0 < (warp + 1) * ROWS; i0 += 4) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int k = 0; k < DK; k += 4) {
                const float4 rv = *reinterpret_cast<const float4*>(Rl + k);
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    const float4 sv = __ldg(reinterpret_cast<const float4*>(S0h + (long long)(i0 + rr) * DK + k));
                    acc[rr] = fmaf(sv.x, rv.x, acc[rr]); acc[rr] = fmaf(sv.y, rv.y, acc[rr]);
                    acc[rr] = fmaf(sv.z, rv.z, acc[rr]); acc[rr] = fmaf(sv.w, rv.w, acc[rr]);
                }
            }
            float4* cp = reinterpret_cast<float4*>(C_s + lane * CP + i0);
            float4 c4 = *cp;
            c4.x += acc[0]; c4.y += acc[1]; c4.z += acc[2]; c4.w += acc[3];
            *cp = c4;
        }
    }
    __syncthreads();

    if (active) {
        OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + b) * Hv + hv) * DV;
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            float x[VEC];
#pragma unroll
            for (int e = 0; e < VEC; e += 4) {
                const float4 t = *reinterpret_cast<const float4*>(C_s + grp * CP + (c * G + g) * VEC + e);
                x[e] = t.x; x[e + 1] = t.y; x[e + 2] = t.z; x[e + 3] = t.w;
            }
            store_out<OutT, VEC>(out + (c * G + g) * VEC, x);
        }
    }
}

// One thread per 16-byte chunk: keys to the key heads' plane, values and gates to the value heads' planes, bit for bit.
__global__ void append_grouped_kernel(const char* __restrict__ k, const char* __restrict__ v, const float* __restrict__ alpha,
                                      const float* __restrict__ beta, char* __restrict__ kplane, char* __restrict__ vplane,
                                      float2* __restrict__ gates, long long arena_slots, int W, int Hk, int g, int kbytes,
                                      int vbytes, BatchBases bases) {
    const int req = blockIdx.y, Hv = Hk * g;
    const int kch = kbytes / 16, vch = vbytes / 16;
    const long long per_beam = (long long)Hk * kch + (long long)Hv * vch + Hv;   // k chunks, v chunks, gate pairs
    const long long total = (long long)W * per_beam;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(i / per_beam);
        long long j = i - (long long)b * per_beam;
        const long long slot = bases.base[req] + b;
        if (j < (long long)Hk * kch) {
            const int h = (int)(j / kch), c = (int)(j - (long long)h * kch);
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(k + (((long long)req * W + b) * Hk + h) * kbytes) + c);
            reinterpret_cast<uint4*>(kplane + ((long long)h * arena_slots + slot) * kbytes)[c] = x;
            continue;
        }
        j -= (long long)Hk * kch;
        if (j < (long long)Hv * vch) {
            const int h = (int)(j / vch), c = (int)(j - (long long)h * vch);
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(v + (((long long)req * W + b) * Hv + h) * vbytes) + c);
            reinterpret_cast<uint4*>(vplane + ((long long)h * arena_slots + slot) * vbytes)[c] = x;
            continue;
        }
        const int h = (int)(j - (long long)Hv * vch);
        const long long in = ((long long)req * W + b) * Hv + h;
        gates[(long long)h * arena_slots + slot] = make_float2(__ldg(alpha + in), __ldg(beta + in));
    }
}

template <int DK, int DV, typename T, typename OutT>
cudaError_t launch_one(const GroupedArgs& a, cudaStream_t stream) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int G = (DK / VEC >= 8 && DV / VEC >= 8) ? 8 : 4;
    auto kern = decode_grouped_kernel<DK, DV, T, OutT, G>;
    const size_t smem = sizeof(float) * NB * ((DK + 4) + (DV + 4));
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((a.W + NB - 1) / NB, a.Hk * a.g, a.req_count);
    kern<<<grid, NB * G, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int DK, int DV>
cudaError_t launch_dims(const GroupedArgs& a, int32_t rec_dtype, int32_t out_dtype, cudaStream_t stream) {
    if (rec_dtype == ONELA_DTYPE_BF16) {
        return out_dtype == ONELA_DTYPE_BF16 ? launch_one<DK, DV, __nv_bfloat16, __nv_bfloat16>(a, stream)
                                             : launch_one<DK, DV, __nv_bfloat16, float>(a, stream);
    }
    return out_dtype == ONELA_DTYPE_BF16 ? launch_one<DK, DV, float, __nv_bfloat16>(a, stream)
                                         : launch_one<DK, DV, float, float>(a, stream);
}

}  // namespace

bool decode_grouped_supported(int32_t dk, int32_t dv) {
    return (dk == 64 && dv == 64) || (dk == 128 && dv == 128) || (dk == 128 && dv == 256);
}

cudaError_t launch_decode_grouped(const GroupedArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                                  cudaStream_t stream) {
    if (dk == 64 && dv == 64) return launch_dims<64, 64>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 128) return launch_dims<128, 128>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 256) return launch_dims<128, 256>(a, rec_dtype, out_dtype, stream);
    return cudaErrorInvalidValue;
}

cudaError_t launch_append_grouped(const void* k, const void* v, const float* alpha, const float* beta, char* kplane,
                                  char* vplane, float2* gates, long long arena_slots, int32_t req_count, int32_t W,
                                  int32_t Hk, int32_t g, int32_t dk, int32_t dv, int32_t elem_bytes, const BatchBases& bases,
                                  cudaStream_t stream) {
    const long long per_beam = (long long)Hk * (dk * elem_bytes / 16) + (long long)Hk * g * (dv * elem_bytes / 16) + Hk * g;
    const long long total = (long long)W * per_beam;
    const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
    append_grouped_kernel<<<dim3(blocks, req_count), 256, 0, stream>>>(
        static_cast<const char*>(k), static_cast<const char*>(v), alpha, beta, kplane, vplane, gates, arena_slots, W, Hk, g,
        dk * elem_bytes, dv * elem_bytes, bases);
    return cudaGetLastError();
}

}  // namespace onela
