// Fused decode kernel for B200 (sm_100a): dk = dv = 128, bf16 records.
//
// Persistent CTAs (two per SM) walk a contiguous range of work items (request, head, tile of 32 beams).
// For every tile:
//   1. fold  - a group of 8 lanes owns one (beam, head) unit and folds its query through the unit's
//              records newest -> oldest (c = k.r; corr += beta c v; r -= beta c k, decay kept as a scalar).
//              Records are read with coalesced 16-byte read-only loads (8 lanes cover 128 contiguous
//              bytes), one level prefetched ahead; shared ancestors are served by L1/L2.
//   2. meet  - the 32 folded queries are written to shared memory as a K-major, 128-byte-swizzled
//              operand; the head's S_0 (pre-swizzled, TF32-rounded image in the store) arrives by ONE
//              64 KiB bulk async copy that was issued before the fold and stays resident while
//              consecutive tiles belong to the same head; one thread issues 16 tcgen05.mma
//              (kind::tf32, M = dv = 128, N = 32 beams, K = 8) accumulating fp32 in tensor memory.
//   3. finish- tcgen05.ld brings the [dv x 32] accumulator back, it is transposed through shared
//              memory, the fold groups add their corr registers and store coalesced rows.
// Every wait is bounded: on expiry the CTA records ONELA_E_TIMEOUT in the status word, stops taking
// tiles, releases its tensor memory and returns.
#include <cstdio>

#include "onela_internal.h"
#include "onela_layout.cuh"

namespace onela {

namespace {

constexpr int NT = 32;              // beams per tile (= MMA N)
constexpr int THREADS = NT * 8;     // 8 lanes per unit
constexpr int DK = 128, DV = 128;
constexpr int S0_BYTES = DV * DK * 4;          // 65536
constexpr int R_KB_STRIDE = NT * 128;          // bytes between K blocks of the R operand
constexpr int R_BYTES = 4 * R_KB_STRIDE;       // 16384
constexpr int OP = DV + 4;                     // pitch (floats) of the transposed accumulator
constexpr int O_BYTES = NT * OP * 4;           // 16896
constexpr int SMEM_BYTES = S0_BYTES + R_BYTES + O_BYTES + 64 + 1024;  // + barriers + alignment slack
constexpr uint32_t TMEM_COLS = 32;
constexpr int WAIT_LIMIT = 1 << 20;

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
// Instruction descriptor: D fp32, A and B TF32, both K-major, M = 128, N = NT.
constexpr uint32_t IDESC = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
        : "memory");
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

struct Rec {           // one lane's share of a record: 2 x 8 elements of k, 2 x 8 of v, and the gates
    uint4 k0, k1, v0, v1;
    float2 gate;
};

__device__ __forceinline__ Rec load_rec(const char* kv, const float2* gates, long long row, int g) {
    const uint4* p = reinterpret_cast<const uint4*>(kv + row * ((DK + DV) * 2)) + g;
    Rec r;
    r.k0 = __ldg(p);
    r.k1 = __ldg(p + 8);
    r.v0 = __ldg(p + 16);
    r.v1 = __ldg(p + 24);
    r.gate = __ldg(gates + row);
    return r;
}
// two packed bf16 -> float2 {element 0, element 1}, exactly
__device__ __forceinline__ float2 up2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void unpack8(const uint4& x, float2* o) {
    o[0] = up2(x.x); o[1] = up2(x.y); o[2] = up2(x.z); o[3] = up2(x.w);
}

// One fold step on this lane's 16 elements (packed fp32x2 FMAs), with the 8-lane dot reduction:
//   c~ = k . r~ ;  corr += (decay beta c~) v ;  r~ -= (beta c~) k ;  decay *= alpha
__device__ __forceinline__ void fold_step(const Rec& rec, float2* r, float2* corr, float& decay) {
    float2 kx[8];
    unpack8(rec.k0, kx);
    unpack8(rec.k1, kx + 4);
    float2 d0 = make_float2(0.f, 0.f), d1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
        d0 = __ffma2_rn(kx[e], r[e], d0);
        d1 = __ffma2_rn(kx[e + 1], r[e + 1], d1);
    }
    float dot = (d0.x + d0.y) + (d1.x + d1.y);
    dot += __shfl_xor_sync(0xffffffffu, dot, 4);
    dot += __shfl_xor_sync(0xffffffffu, dot, 2);
    dot += __shfl_xor_sync(0xffffffffu, dot, 1);
    const float bc = rec.gate.y * dot;
    const float wv = decay * bc;
    const float2 nbc2 = make_float2(-bc, -bc), wv2 = make_float2(wv, wv);
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = __ffma2_rn(kx[e], nbc2, r[e]);
    float2 vx[8];
    unpack8(rec.v0, vx);
    unpack8(rec.v1, vx + 4);
#pragma unroll
    for (int e = 0; e < 8; ++e) corr[e] = __ffma2_rn(vx[e], wv2, corr[e]);
    decay *= rec.gate.x;
}

template <typename OutT>
__global__ void __launch_bounds__(THREADS, 2) decode_sm100_kernel(const DecodeArgs a, int total_tiles, int tiles_per_pair) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t s0_addr = base, r_addr = base + S0_BYTES;
    uint8_t* R_s = smem + S0_BYTES;
    float* O_s = reinterpret_cast<float*>(smem + S0_BYTES + R_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S0_BYTES + R_BYTES + O_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
    const uint32_t bar_s0 = smem_u32(bars), bar_mma = smem_u32(bars + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = tid >> 3, g = tid & 7;

    if (tid == 0) {
        mbar_init(bar_s0, 1);
        mbar_init(bar_mma, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // contiguous range of tiles for this CTA
    const int t_begin = (int)(((long long)blockIdx.x * total_tiles) / gridDim.x);
    const int t_end = (int)(((long long)(blockIdx.x + 1) * total_tiles) / gridDim.x);

    const char* kv = a.kv;
    const __nv_bfloat16* qbase = static_cast<const __nv_bfloat16*>(a.q);
    int cur_pair = -1;
    uint32_t s0_phase = 0, mma_phase = 0;
    int failed = 0;

    // Decompose a tile index and fetch what its fold needs first: the query and the beam's own record.
    struct TileHead {
        int req, h, b, bb;
        bool active;
        uint4 q0, q1;
        Rec own;
    };
    auto open_tile = [&](int tile) {
        TileHead t;
        const int pair = tile / tiles_per_pair, tb = tile - pair * tiles_per_pair;
        t.req = pair / a.H;
        t.h = pair - t.req * a.H;
        t.b = tb * NT + grp;
        t.active = t.b < a.W;
        t.bb = t.active ? t.b : a.W - 1;   // idle groups shadow a live beam: loads and shuffles stay uniform
        const uint4* qp = reinterpret_cast<const uint4*>(qbase + (((long long)t.req * a.W + t.bb) * a.H + t.h) * DK) + g;
        t.q0 = __ldg(qp);
        t.q1 = __ldg(qp + 8);
        t.own = load_rec(kv, a.gates, (long long)t.h * a.arena_slots + a.bases.base[t.req] + t.bb, g);
        return t;
    };

#ifdef ONELA_TIMING
    long long tph[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    long long tk = clock64();
    const long long tstart = tk;
#define ONELA_TICK(i) { const long long now = clock64(); tph[i] += now - tk; tk = now; }
#else
#define ONELA_TICK(i)
#endif
    TileHead th = open_tile(t_begin);
    for (int tile = t_begin; tile < t_end; ++tile) {
        const int req = th.req, h = th.h, b = th.b, bb = th.bb;
        const bool active = th.active;
        const int pair = req * a.H + h;
        bool s0_pending = false;
        if (pair != cur_pair) {
            cur_pair = pair;
            s0_pending = true;
            if (tid == 0) {   // every MMA that read the previous image has completed (bar_mma was waited on)
                mbar_expect_tx(bar_s0, S0_BYTES);
                bulk_load(s0_addr, a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK), S0_BYTES, bar_s0);
            }
        }

        // ---- 1. fold ------------------------------------------------------------------------------
        const long long plane_row0 = (long long)h * a.arena_slots;
        const int32_t* table = a.table + req * a.table_req_stride + bb;
        const int old = a.depth - 1;          // records older than the beam's own: levels old-1 .. 0
        // lane g keeps the slot of level g (levels 0..7); deeper chains read the rest on demand
        const int32_t my_slot = (g < old) ? __ldg(table + (long long)g * a.max_beam) : 0;
        auto slot_of = [&](int level) -> int32_t {
            const int32_t s = __shfl_sync(0xffffffffu, my_slot, level & 7, 8);
            return level < 8 ? s : __ldg(table + (long long)level * a.max_beam);
        };
        auto load_level = [&](int level) { return load_rec(kv, a.gates, plane_row0 + slot_of(level), g); };

        float2 r[8], corr[8];
        unpack8(th.q0, r);
        unpack8(th.q1, r + 4);
#pragma unroll
        for (int e = 0; e < 8; ++e) corr[e] = make_float2(0.f, 0.f);
        float decay = 1.f;

#ifndef ONELA_PF1
        // three record buffers rotate: while one is folded the next two are in flight
        Rec A = th.own, B, C;
        int level = old;                       // level being folded; level == old is the own record
        if (level >= 1) B = load_level(level - 1);
        while (true) {
            if (level >= 2) C = load_level(level - 2);
            fold_step(A, r, corr, decay);
            if (--level < 0) break;
            if (level >= 2) A = load_level(level - 2);
            fold_step(B, r, corr, decay);
            if (--level < 0) break;
            if (level >= 2) B = load_level(level - 2);
            fold_step(C, r, corr, decay);
            if (--level < 0) break;
        }
#else
        // two record buffers: while one is folded the next is in flight
        Rec A = th.own, B;
        int level = old;
        while (true) {
            if (level >= 1) B = load_level(level - 1);
            fold_step(A, r, corr, decay);
            if (--level < 0) break;
            if (level >= 1) A = load_level(level - 1);
            fold_step(B, r, corr, decay);
            if (--level < 0) break;
        }
#endif

        ONELA_TICK(0)   // fold

        // ---- 2. meet S_0 ----------------------------------------------------------------------------
        // lane g holds elements [8g, 8g+8) and [64+8g, 64+8g+8) of the folded query of beam `grp`
        {
            const int sw = grp & 7;
            const float2 dc = make_float2(decay, decay);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int kb = 2 * c + (g >> 2);            // K block of 32 floats
                const int ch = 2 * (g & 3);                 // first of two 16-byte chunks inside the 128-byte row
                uint8_t* row = R_s + kb * R_KB_STRIDE + grp * 128;
                float2 x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = __fmul2_rn(r[4 * c + e], dc);
                *reinterpret_cast<float4*>(row + (((ch) ^ sw) << 4)) =
                    make_float4(round_tf32(x[0].x), round_tf32(x[0].y), round_tf32(x[1].x), round_tf32(x[1].y));
                *reinterpret_cast<float4*>(row + (((ch + 1) ^ sw) << 4)) =
                    make_float4(round_tf32(x[2].x), round_tf32(x[2].y), round_tf32(x[3].x), round_tf32(x[3].y));
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        ONELA_TICK(1)   // R write
        if (__syncthreads_or(failed)) break;
        ONELA_TICK(2)   // barrier A
        // The next tile's query and own record start their trip now and land during the MMA and the
        // epilogue.  (Issued after the proxy fence above: that fence waits for loads in flight.)
#ifndef ONELA_NO_XTILE
        if (tile + 1 < t_end) th = open_tile(tile + 1);
#endif
        ONELA_TICK(6)   // open next tile

        if (tid == 0) {
            bool ok = true;
            if (s0_pending) ok = mbar_wait(bar_s0, s0_phase);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (ok) {
#pragma unroll
                for (int kb = 0; kb < 4; ++kb)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_tf32(tmem_base, umma_desc(s0_addr + kb * (DV * 128) + ks * 32),
                                  umma_desc(r_addr + kb * R_KB_STRIDE + ks * 32), (kb | ks) ? 1u : 0u);
            } else {
                failed = 1;
            }
            umma_commit(bar_mma);   // arrives when the MMAs above (if any) have completed
        }
        if (s0_pending) s0_phase ^= 1;
        ONELA_TICK(7)   // S0 wait + MMA issue (thread 0)

        // ---- 3. finish --------------------------------------------------------------------------------
        if (!mbar_wait(bar_mma, mma_phase)) failed = 1;
        mma_phase ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        ONELA_TICK(3)   // MMA issue + wait
        {
            // warp w reads accumulator rows (dv) 32*(w&3) + lane, beams 16*(w>>2) .. +16
            const int col0 = (warp >> 2) * 16;
            uint32_t v[16];
            tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)col0, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int i = (warp & 3) * 32 + lane;
#pragma unroll
            for (int j = 0; j < 16; ++j) O_s[(col0 + j) * OP + i] = __uint_as_float(v[j]);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        if (__syncthreads_or(failed)) break;
        ONELA_TICK(4)   // tmem ld + transpose + barrier B

        if (active) {
            OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + b) * a.H + h) * DV;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int e0 = (c * 8 + g) * 8;
                const float4 x0 = *reinterpret_cast<const float4*>(O_s + grp * OP + e0);
                const float4 x1 = *reinterpret_cast<const float4*>(O_s + grp * OP + e0 + 4);
                const float2* cc = corr + 4 * c;
                float o[8] = {x0.x + cc[0].x, x0.y + cc[0].y, x0.z + cc[1].x, x0.w + cc[1].y,
                              x1.x + cc[2].x, x1.y + cc[2].y, x1.z + cc[3].x, x1.w + cc[3].y};
                store8<OutT>(out + e0, o);
            }
        }
#ifdef ONELA_NO_XTILE
        if (tile + 1 < t_end) th = open_tile(tile + 1);
#endif
        ONELA_TICK(5)   // store
    }
#ifdef ONELA_TIMING
    if ((tid == 0 || tid == 255) && (blockIdx.x == 0 || blockIdx.x == 150 || blockIdx.x == gridDim.x - 1))
        printf("cta %d tid %d depth %d tiles %d total %lld | fold %lld Rwrite %lld barA %lld mmawait %lld ld+barB %lld store %lld open %lld issue %lld\n",
               (int)blockIdx.x, tid, a.depth, t_end - t_begin, clock64() - tstart, tph[0], tph[1], tph[2], tph[3], tph[4], tph[5], tph[6], tph[7]);
#endif

    if (failed && tid == 0) {
        if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)blockIdx.x;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

template <typename OutT>
cudaError_t launch_t(const DecodeArgs& a, cudaStream_t stream) {
    auto kern = decode_sm100_kernel<OutT>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int tiles_per_pair = (a.W + NT - 1) / NT;
    const int total_tiles = a.req_count * a.H * tiles_per_pair;
    const int grid = total_tiles < 2 * sm_count() ? total_tiles : 2 * sm_count();
    kern<<<grid, THREADS, SMEM_BYTES, stream>>>(a, total_tiles, tiles_per_pair);
    return cudaGetLastError();
}

}  // namespace

bool decode_sm100_supported(int32_t dk, int32_t dv, int32_t rec_dtype) {
    return dk == 128 && dv == 128 && rec_dtype == ONELA_DTYPE_BF16;
}

cudaError_t launch_decode_sm100(const DecodeArgs& a, int32_t out_dtype, cudaStream_t stream) {
    return out_dtype == ONELA_DTYPE_BF16 ? launch_t<__nv_bfloat16>(a, stream) : launch_t<float>(a, stream);
}

}  // namespace onela
