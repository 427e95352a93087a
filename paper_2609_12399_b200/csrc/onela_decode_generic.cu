// CUDA-core decode kernel for every supported (dk, dv, dtype): the product path for shapes the
// tensor-core kernel does not cover (e.g. dk = dv = 32 fp32) and the A/B partner of that kernel.
//
// One CTA = (request, head, tile of 32 beams).  A group of G lanes owns one (beam, head) unit and
// folds its query through the unit's records, newest first (see onela.h):
//      c = k_j . r ;  corr += beta_j c v_j ;  r <- alpha_j (r - beta_j c k_j)
// with the decay kept as a running scalar (r = a * r~, a = prod alpha) so each record costs one dot,
// two axpys and a log2(G)-step shuffle reduction.  The folded queries of the tile then meet the head's
// S_0 in a [dv x dk] . [dk x 32] product on the FMA pipes: lane = beam, each warp a band of rows,
// S_0 rows read as warp-uniform (broadcast) 16-byte loads, R from padded shared memory.
#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {

namespace {

constexpr int NB = 32;  // beams per tile

template <int DK, int DV, typename T, typename OutT, int G>
__global__ void __launch_bounds__(NB* G) decode_generic_kernel(const DecodeArgs a) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int CK = DK / (G * VEC), CV = DV / (G * VEC);  // 16-byte chunks per lane
    static_assert(CK >= 1 && CV >= 1 && DK % (G * VEC) == 0 && DV % (G * VEC) == 0, "lane mapping");
    static_assert((DV / G) % 4 == 0, "row bands of the contraction");
    constexpr int RP = DK + 4, CP = DV + 4;  // padded pitches (floats): conflict-free 16-byte accesses
    extern __shared__ __align__(16) float smem[];
    float* R_s = smem;             // [NB][RP]  folded queries
    float* C_s = smem + NB * RP;   // [NB][CP]  corr, then the finished outputs

    const int tile = blockIdx.x, h = blockIdx.y, req = blockIdx.z;
    const int grp = threadIdx.x / G, g = threadIdx.x % G;
    const int b = tile * NB + grp;
    const bool active = b < a.W;
    const int bb = active ? b : a.W - 1;  // idle groups shadow a live beam so loads and shuffles stay uniform

    const T* q = static_cast<const T*>(a.q) + (((long long)req * a.W + bb) * a.H + h) * DK;
    const int32_t* table = a.table + req * a.table_req_stride;
    const long long plane_row0 = (long long)h * a.arena_slots;
    const T* kv = reinterpret_cast<const T*>(a.kv);

    float r[CK * VEC], corr[CV * VEC];
#pragma unroll
    for (int c = 0; c < CK; ++c) Vec16<T>::load(q + (c * G + g) * VEC, r + c * VEC);
#pragma unroll
    for (int e = 0; e < CV * VEC; ++e) corr[e] = 0.f;

    float decay = 1.f;  // a = product of the alphas already passed
    for (int level = a.depth - 1; level >= 0; --level) {
        const int32_t slot = (level == a.depth - 1) ? a.bases.base[req] + bb
                                                    : __ldg(table + (long long)level * a.max_beam + bb);
        const long long row = plane_row0 + slot;
        const T* rec = kv + row * (DK + DV);
        const float2 gate = __ldg(a.gates + row);
        float kx[CK * VEC];
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            Vec16<T>::load(rec + (c * G + g) * VEC, kx + c * VEC);
#pragma unroll
            for (int e = 0; e < VEC; ++e) dot = fmaf(kx[c * VEC + e], r[c * VEC + e], dot);
        }
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        const float bc = gate.y * dot;        // beta_j * (k_j . r~_j)
        const float wv = decay * bc;          // beta_j * c_j with c_j = a_j (k_j . r~_j)
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            float vx[VEC];
            Vec16<T>::load(rec + DK + (c * G + g) * VEC, vx);
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
        const float* S0h = a.s0 + req * a.s0_req_stride + (long long)h * DV * DK;
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
                    acc[rr] = fmaf(sv.x, rv.x, acc[rr]);
                    acc[rr] = fmaf(sv.y, rv.y, acc[rr]);
                    acc[rr] = fmaf(sv.z, rv.z, acc[rr]);
                    acc[rr] = fmaf(sv.w, rv.w, acc[rr]);
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
        OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + b) * a.H + h) * DV;
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

template <int DK, int DV, typename T, typename OutT>
cudaError_t launch_one(const DecodeArgs& a, cudaStream_t stream) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int G = (DK / VEC >= 8 && DV / VEC >= 8) ? 8 : 4;
    auto kern = decode_generic_kernel<DK, DV, T, OutT, G>;
    const size_t smem = sizeof(float) * NB * ((DK + 4) + (DV + 4));
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((a.W + NB - 1) / NB, a.H, a.req_count);
    kern<<<grid, NB * G, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int DK, int DV>
cudaError_t launch_dims(const DecodeArgs& a, int32_t rec_dtype, int32_t out_dtype, cudaStream_t stream) {
    if (rec_dtype == ONELA_DTYPE_BF16) {
        return out_dtype == ONELA_DTYPE_BF16 ? launch_one<DK, DV, __nv_bfloat16, __nv_bfloat16>(a, stream)
                                             : launch_one<DK, DV, __nv_bfloat16, float>(a, stream);
    }
    return out_dtype == ONELA_DTYPE_BF16 ? launch_one<DK, DV, float, __nv_bfloat16>(a, stream)
                                         : launch_one<DK, DV, float, float>(a, stream);
}

}  // namespace

bool decode_generic_supported(int32_t dk, int32_t dv, int32_t rec_dtype) {
    (void)rec_dtype;
    return (dk == 32 && dv == 32) || (dk == 64 && dv == 64) || (dk == 128 && dv == 128) ||
           (dk == 128 && dv == 256) || (dk == 256 && dv == 256) || (dk == 128 && dv == 512) || (dk == 256 && dv == 512);
}

cudaError_t launch_decode_generic(const DecodeArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype,
                                  int32_t out_dtype, bool* supported, cudaStream_t stream) {
    *supported = true;
    if (dk == 32 && dv == 32) return launch_dims<32, 32>(a, rec_dtype, out_dtype, stream);
    if (dk == 64 && dv == 64) return launch_dims<64, 64>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 128) return launch_dims<128, 128>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 256) return launch_dims<128, 256>(a, rec_dtype, out_dtype, stream);
    if (dk == 256 && dv == 256) return launch_dims<256, 256>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 512) return launch_dims<128, 512>(a, rec_dtype, out_dtype, stream);
    if (dk == 256 && dv == 512) return launch_dims<256, 512>(a, rec_dtype, out_dtype, stream);
    *supported = false;
    return cudaErrorInvalidValue;
}

}  // namespace onela
