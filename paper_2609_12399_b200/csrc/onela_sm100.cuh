// PTX wrappers and fold primitives shared by the sm_100a decode kernels (dk = dv = 128, bf16 records):
// mbarriers, bulk async copies, tcgen05 MMA / tensor-memory access, and the per-lane fold step.
#pragma once

#include <cuda_fp16.h>

#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {
namespace sm100 {

constexpr int DK = 128, DV = 128;
constexpr int REC_BYTES = (DK + DV) * 2;       // 512: k | v in bf16
#ifndef ONELA_WAIT_LIMIT
#define ONELA_WAIT_LIMIT (1 << 20)
#endif
constexpr int WAIT_LIMIT = ONELA_WAIT_LIMIT;     // probes of a barrier before a wait gives up (the test-hooks build uses fewer)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the phase did not complete within WAIT_LIMIT probes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Named barrier over `count` threads that also ORs a predicate across them.
__device__ __forceinline__ int bar_or(int id, int count, int pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(pred), "r"(id), "r"(count)
        : "memory");
    return (int)out;
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);       // start address, 16-byte units
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                            // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
    return d;
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

// Instruction descriptor: D fp32, A and B fp16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_f16(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// tcgen05.mma, fp16 operands (K = 16 per instruction), A in tensor memory: lane = row, two K elements per 32-bit column.
__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// tcgen05.mma, fp16 operands, A and B both from shared memory (K-major, 128-byte swizzle)
__device__ __forceinline__ void umma_f16_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// two fp32 -> packed fp16 (element 0 in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    const __half2 t = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
// Write 16 consecutive columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        :
        : "r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
// Write 8 consecutive columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 :
                 : "r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
// The power of two that brings a positive magnitude m into [2^target, 2^(target + 1)), and its reciprocal; both 1 when
// m is zero, subnormal, infinite, NaN or too small for the reciprocal to be a normal number.  Used to keep fp16
// operands inside the format's normal range whatever the scale of the caller's data (multiplying by them is exact).
__device__ __forceinline__ void pow2_scale(float m, int target, float& scale, float& inv) {
    const int eb = (int)(__float_as_uint(m) >> 23) & 255;          // biased exponent (m >= 0)
    const bool ok = eb > target + 1 && eb < 255;
    scale = ok ? __uint_as_float((uint32_t)(254 + target - eb) << 23) : 1.f;
    inv = ok ? __uint_as_float((uint32_t)(eb - target) << 23) : 1.f;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
template <typename OutT>
__device__ __forceinline__ void store8(OutT* p, const float* x);
template <>
__device__ __forceinline__ void store8<float>(float* p, const float* x) {
    reinterpret_cast<float4*>(p)[0] = make_float4(x[0], x[1], x[2], x[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(x[4], x[5], x[6], x[7]);
}
template <>
__device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* p, const float* x) {
    *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]), pack_bf16x2(x[4], x[5]),
                                              pack_bf16x2(x[6], x[7]));
}

// One lane's share of a record: NCH x 8 elements of k, NCH x 8 of v (packed bf16), and the gates.
template <int NCH>
struct Rec {
    uint4 k[NCH], v[NCH];
    float2 gate;
};

// two packed bf16 -> float2 {element 0, element 1}, exactly
__device__ __forceinline__ float2 up2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void unpack8(const uint4& x, float2* o) {
    o[0] = up2(x.x); o[1] = up2(x.y); o[2] = up2(x.z); o[3] = up2(x.w);
}

// LPU lanes share one (beam, head) unit; lane g owns the 16-byte chunks c*LPU + g (c < NCH) of every
// 256-byte vector, i.e. elements [(c*LPU + g)*8, +8): LPU consecutive lanes cover contiguous memory.
template <int LPU>
struct Lanes {
    static constexpr int NCH = 16 / LPU;     // 16-byte chunks per lane per 128-element bf16 vector
    static constexpr int NP2 = 4 * NCH;      // float2 pairs per lane
    using R = Rec<NCH>;

    static __device__ __forceinline__ R load_global(const char* kv, const float2* gates, long long row, int g) {
        const uint4* p = reinterpret_cast<const uint4*>(kv + row * REC_BYTES) + g;
        R r;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            r.k[c] = __ldg(p + c * LPU);
            r.v[c] = __ldg(p + 16 + c * LPU);
        }
        r.gate = __ldg(gates + row);
        return r;
    }
    static __device__ __forceinline__ R load_shared(const uint8_t* stage, const float2* gates_s, int idx, int g) {
        const uint4* p = reinterpret_cast<const uint4*>(stage + idx * REC_BYTES) + g;
        R r;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            r.k[c] = p[c * LPU];
            r.v[c] = p[16 + c * LPU];
        }
        r.gate = gates_s[idx];
        return r;
    }
    // One fold step on this lane's elements (packed fp32x2 FMAs), with the LPU-lane dot reduction:
    //   c~ = k . r~ ;  corr += (decay beta c~) v ;  r~ -= (beta c~) k ;  decay *= alpha
    // REPLAY (records (alpha, delta, k), Eq. 3): the vector is not changed, the record's second half is the stored
    // update vector delta, taken with the weight decay * (k . r):   corr += (decay c~) delta ;  decay *= alpha
    template <bool REPLAY = false>
    static __device__ __forceinline__ void fold_step(const R& rec, float2* r, float2* corr, float& decay) {
        float2 kx[NP2];
#pragma unroll
        for (int c = 0; c < NCH; ++c) unpack8(rec.k[c], kx + 4 * c);
        float2 d0 = make_float2(0.f, 0.f), d1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < NP2; e += 2) {
            d0 = __ffma2_rn(kx[e], r[e], d0);
            d1 = __ffma2_rn(kx[e + 1], r[e + 1], d1);
        }
        float dot = (d0.x + d0.y) + (d1.x + d1.y);
#pragma unroll
        for (int o = LPU / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        const float bc = REPLAY ? dot : rec.gate.y * dot;
        const float wv = decay * bc;
        const float2 nbc2 = make_float2(-bc, -bc), wv2 = make_float2(wv, wv);
        if (!REPLAY) {
#pragma unroll
            for (int e = 0; e < NP2; ++e) r[e] = __ffma2_rn(kx[e], nbc2, r[e]);
        }
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            float2 vx[4];
            unpack8(rec.v[c], vx);
#pragma unroll
            for (int e = 0; e < 4; ++e) corr[4 * c + e] = __ffma2_rn(vx[e], wv2, corr[4 * c + e]);
        }
        decay *= rec.gate.x;
    }
    // Single-buffered chain: fetch a record, fold it (for sources whose latency is short, or to save registers).
    template <bool REPLAY = false, class LoadFn>
    static __device__ __forceinline__ void fold_chain_simple(const R& first, int hi, int lo, LoadFn load, float2* r,
                                                             float2* corr, float& decay) {
        fold_step<REPLAY>(first, r, corr, decay);
        for (int level = hi; level >= lo; --level) {
            const R rec = load(level);
            fold_step<REPLAY>(rec, r, corr, decay);
        }
    }
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}


}  // namespace sm100
}  // namespace onela
