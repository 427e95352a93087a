// Forward projection replay over (alpha, delta, k) transition records: the record format and the replay order
// of Section 3.2 (Eq. 2-4), as a CUDA-core kernel.  Selected by ONELA_FLAG_GTR_DELTA; the default path keeps raw
// (k, v, alpha, beta) records and folds the query backward (onela_decode_sm100.cu, onela_decode_generic.cu).
//
// One launch = append + decode of one layer (the update vector delta_t needs the key projection of the parent
// state, so the record can only be produced where the replay runs).  One CTA = (request, head, tile of 32
// beams).  A group of G lanes owns one (beam, head) unit:
//   1. the tile's queries and current keys go to shared memory and meet the head's S_0 in two
//      [dv x dk] . [dk x 32] products on the FMA pipes (lane = beam, each warp a band of rows, S_0 rows read as
//      warp-uniform 16-byte loads):  u_q = S_0 q_t,  u_k = S_0 k_t                                   (Eq. 3, j = -1)
//   2. replay, oldest ancestor first:  u_q <- alpha_j u_q + delta_j (k_j . q_t),
//                                      u_k <- alpha_j u_k + delta_j (k_j . k_t)                      (Eq. 3)
//      the two dot products of a level do not depend on the level before it; only the axpys chain.
//   3. delta_t = beta_t (v_t - alpha_t u_k);  o_t = alpha_t u_q + delta_t (k_t . q_t)                (Eq. 4)
//      the record (k_t, delta_t in the record dtype, alpha_t) goes to the beam's arena slot, o_t to the output.
// The stored delta is rounded to the record dtype (bf16 in the benchmark shapes); later steps replay the rounded
// value, which is where this variant's extra error against the exact recurrence comes from.
#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {

namespace {

constexpr int NB = 32;  // beams per tile

// N consecutive elements (one 16-byte vector of T) from fp32
template <typename T>
__device__ __forceinline__ void store_vec(T* p, const float* x);
template <>
__device__ __forceinline__ void store_vec<float>(float* p, const float* x) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
template <>
__device__ __forceinline__ void store_vec<__nv_bfloat16>(__nv_bfloat16* p, const float* x) {
    *reinterpret_cast<uint4*>(p) = make_uint4(pack2(x[0], x[1]), pack2(x[2], x[3]), pack2(x[4], x[5]), pack2(x[6], x[7]));
}
template <int DK, int DV, typename T, typename OutT, int G>
__global__ void __launch_bounds__(NB* G) decode_gtr_kernel(const DecodeArgs a) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int CK = DK / (G * VEC), CV = DV / (G * VEC);  // 16-byte chunks per lane
    static_assert(CK >= 1 && CV >= 1 && DK % (G * VEC) == 0 && DV % (G * VEC) == 0, "lane mapping");
    static_assert((DV / G) % 4 == 0, "row bands of the contraction");
    constexpr int RP = DK + 4, CP = DV + 4;  // padded pitches (floats): conflict-free 16-byte accesses
    extern __shared__ __align__(16) float smem[];
    float* Q_s = smem;                  // [NB][RP]  queries
    float* K_s = Q_s + NB * RP;         // [NB][RP]  current keys
    float* Uq_s = K_s + NB * RP;        // [NB][CP]  S_0 q
    float* Uk_s = Uq_s + NB * CP;       // [NB][CP]  S_0 k

    const int tile = blockIdx.x, h = blockIdx.y, req = blockIdx.z;
    const int grp = threadIdx.x / G, g = threadIdx.x % G;
    const int b = tile * NB + grp;
    const bool active = b < a.W;
    const int bb = active ? b : a.W - 1;  // idle groups shadow a live beam so loads and shuffles stay uniform

    const long long in_row = ((long long)req * a.W + bb) * a.H + h;
    const T* q_in = static_cast<const T*>(a.q) + in_row * DK;
    const T* k_in = static_cast<const T*>(a.k_in) + in_row * DK;
    const T* v_in = static_cast<const T*>(a.v_in) + in_row * DV;
    const int32_t* table = a.table + req * a.table_req_stride;
    const long long plane_row0 = (long long)h * a.arena_slots;
    const T* kv = reinterpret_cast<const T*>(a.kv);

    float q[CK * VEC], kt[CK * VEC];
    float kq = 0.f;                       // k_t . q_t
#pragma unroll
    for (int c = 0; c < CK; ++c) {
        Vec16<T>::load(q_in + (c * G + g) * VEC, q + c * VEC);
        Vec16<T>::load(k_in + (c * G + g) * VEC, kt + c * VEC);
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
            const int o = c * VEC + e;
            *reinterpret_cast<float4*>(Q_s + grp * RP + (c * G + g) * VEC + e) = make_float4(q[o], q[o + 1], q[o + 2], q[o + 3]);
            *reinterpret_cast<float4*>(K_s + grp * RP + (c * G + g) * VEC + e) = make_float4(kt[o], kt[o + 1], kt[o + 2], kt[o + 3]);
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) kq = fmaf(kt[c * VEC + e], q[c * VEC + e], kq);
    }
#pragma unroll
    for (int off = G / 2; off > 0; off >>= 1) kq += __shfl_xor_sync(0xffffffffu, kq, off);
    __syncthreads();

    // u_q[beam][i] = sum_k S0[i][k] q[beam][k], u_k likewise; lane = beam, warp = band of DV/G rows
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const float* S0h = a.s0 + req * a.s0_req_stride + (long long)h * DV * DK;
        const float* Ql = Q_s + lane * RP;
        const float* Kl = K_s + lane * RP;
        constexpr int ROWS = DV / G;
        for (int i0 = warp * ROWS; i0 < (warp + 1) * ROWS; i0 += 4) {
            float aq[4] = {0.f, 0.f, 0.f, 0.f}, ak[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int k = 0; k < DK; k += 4) {
                const float4 qv = *reinterpret_cast<const float4*>(Ql + k);
                const float4 kv4 = *reinterpret_cast<const float4*>(Kl + k);
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    const float4 sv = __ldg(reinterpret_cast<const float4*>(S0h + (long long)(i0 + rr) * DK + k));
                    aq[rr] = fmaf(sv.x, qv.x, aq[rr]); aq[rr] = fmaf(sv.y, qv.y, aq[rr]);
                    aq[rr] = fmaf(sv.z, qv.z, aq[rr]); aq[rr] = fmaf(sv.w, qv.w, aq[rr]);
                    ak[rr] = fmaf(sv.x, kv4.x, ak[rr]); ak[rr] = fmaf(sv.y, kv4.y, ak[rr]);
                    ak[rr] = fmaf(sv.z, kv4.z, ak[rr]); ak[rr] = fmaf(sv.w, kv4.w, ak[rr]);
                }
            }
            *reinterpret_cast<float4*>(Uq_s + lane * CP + i0) = make_float4(aq[0], aq[1], aq[2], aq[3]);
            *reinterpret_cast<float4*>(Uk_s + lane * CP + i0) = make_float4(ak[0], ak[1], ak[2], ak[3]);
        }
    }
    __syncthreads();

    float uq[CV * VEC], uk[CV * VEC];
#pragma unroll
    for (int c = 0; c < CV; ++c)
#pragma unroll
        for (int e = 0; e < VEC; e += 4) {
            const int o = c * VEC + e;
            const float4 x = *reinterpret_cast<const float4*>(Uq_s + grp * CP + (c * G + g) * VEC + e);
            const float4 y = *reinterpret_cast<const float4*>(Uk_s + grp * CP + (c * G + g) * VEC + e);
            uq[o] = x.x; uq[o + 1] = x.y; uq[o + 2] = x.z; uq[o + 3] = x.w;
            uk[o] = y.x; uk[o + 1] = y.y; uk[o + 2] = y.z; uk[o + 3] = y.w;
        }

    // replay the beam's ancestors, oldest first (levels 0 .. depth - 2; the current token is not a record yet)
    for (int level = 0; level < a.depth - 1; ++level) {
        const int32_t slot = __ldg(table + (long long)level * a.max_beam + bb);
        const long long row = plane_row0 + slot;
        const T* rec = kv + row * (DK + DV);
        const float alpha = __ldg(a.gates + row).x;
        float cq = 0.f, ck = 0.f;
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            float kx[VEC];
            Vec16<T>::load(rec + (c * G + g) * VEC, kx);
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                cq = fmaf(kx[e], q[c * VEC + e], cq);
                ck = fmaf(kx[e], kt[c * VEC + e], ck);
            }
        }
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) {
            cq += __shfl_xor_sync(0xffffffffu, cq, off);
            ck += __shfl_xor_sync(0xffffffffu, ck, off);
        }
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            float dx[VEC];
            Vec16<T>::load(rec + DK + (c * G + g) * VEC, dx);
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                uq[c * VEC + e] = fmaf(dx[e], cq, alpha * uq[c * VEC + e]);
                uk[c * VEC + e] = fmaf(dx[e], ck, alpha * uk[c * VEC + e]);
            }
        }
    }

    // the current token: its update vector and the output (Eq. 4); the record goes to the beam's own slot
    const float alpha_t = __ldg(a.alpha_in + in_row), beta_t = __ldg(a.beta_in + in_row);
    const long long own_row = plane_row0 + a.bases.base[req] + bb;
    T* rec_out = reinterpret_cast<T*>(a.kv_out) + own_row * (DK + DV);
    OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + bb) * a.H + h) * DV;
#pragma unroll
    for (int c = 0; c < CV; ++c) {
        float vx[VEC], delta[VEC], o[VEC];
        Vec16<T>::load(v_in + (c * G + g) * VEC, vx);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            delta[e] = beta_t * (vx[e] - alpha_t * uk[c * VEC + e]);
            o[e] = fmaf(delta[e], kq, alpha_t * uq[c * VEC + e]);
        }
        if (active) {
            store_vec<T>(rec_out + DK + (c * G + g) * VEC, delta);
            store_out<OutT, VEC>(out + (c * G + g) * VEC, o);
        }
    }
    if (active) {
#pragma unroll
        for (int c = 0; c < CK; ++c)   // the key, bit for bit
            *reinterpret_cast<uint4*>(rec_out + (c * G + g) * VEC) = __ldg(reinterpret_cast<const uint4*>(k_in + (c * G + g) * VEC));
        if (g == 0) a.gates_out[own_row] = make_float2(alpha_t, beta_t);
    }
}

template <int DK, int DV, typename T, typename OutT>
cudaError_t launch_one(const DecodeArgs& a, cudaStream_t stream) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int G = (DK / VEC >= 8 && DV / VEC >= 8) ? 8 : 4;
    auto kern = decode_gtr_kernel<DK, DV, T, OutT, G>;
    const size_t smem = sizeof(float) * NB * (2 * (DK + 4) + 2 * (DV + 4));
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

cudaError_t launch_decode_gtr(const DecodeArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                              bool* supported, cudaStream_t stream) {
    *supported = true;
    if (dk == 32 && dv == 32) return launch_dims<32, 32>(a, rec_dtype, out_dtype, stream);
    if (dk == 64 && dv == 64) return launch_dims<64, 64>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 128) return launch_dims<128, 128>(a, rec_dtype, out_dtype, stream);
    *supported = false;
    return cudaErrorInvalidValue;
}

}  // namespace onela
