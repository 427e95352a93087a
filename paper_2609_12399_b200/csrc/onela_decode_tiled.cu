// Tiled tcgen05 decode kernel for B200 (sm_100a): the shapes the warp-specialised kernel does not take - key widths
// 64 and 256, value widths 64 to 512, fp32 records at every width, grouped value heads or not (the operator suite of
// Section 4.1).  The chain walk is the CUDA-core one (see onela_decode_generic.cu); what moves to the tensor cores is
// the contraction with S_0, which dominates these shapes (dv x dk multiply-adds per unit against 3 dk per record).
//
// One CTA = (request, value head, tile of 32 beams - 64 at key width 256), 8 lanes per (beam, head) unit.
//   1. Every unit folds its query through its records, newest first:  c = k.r ; corr += beta c v ; r -= beta c k,
//      the decay a running scalar.  corr stays in registers.  With the append fused in, the newest record comes from
//      the caller's tensors and the unit also writes it to its arena slot.
//   2. The folded queries go to shared memory as rows of the MMA's B operand: fp16, K-major, 128-byte swizzle, each row
//      times the power of two that brings its largest element into [2^8, 2^9) (exact; undone after the product).
//   3. Per tile of 128 value rows: the S_0 rows become the A operand the same way (fp16, times the head's power of two
//      kept with the state), dk / 16 MMAs (M = 128, N = beams, K = 16) accumulate S_0 . r~ in tensor memory, and while
//      they run the next tile's A operand is built and the previous tile's accumulator is read back (lane = value
//      row), scaled and added to corr in a shared-memory tile whose rows the units then store as 16-byte vectors.  Two
//      A operands and two accumulators alternate.
// The only wait is for the MMAs' completion; it is bounded, and all threads agree on its outcome before going on
// (ONELA_E_TIMEOUT in the status word otherwise).
#include <mutex>

#include "onela_internal.h"
#include "onela_layout.cuh"
#include "onela_sm100.cuh"

namespace onela {

namespace {

using sm100::bulk_load;
using sm100::idesc_f16;
using sm100::mbar_expect_tx;
using sm100::mbar_init;
using sm100::mbar_wait;
using sm100::pack_f16x2;
using sm100::pow2_scale;
using sm100::smem_u32;
using sm100::tmem_ld16;
using sm100::umma_commit;
using sm100::umma_desc;
using sm100::umma_f16_ss;

constexpr int G = 8;                   // lanes per unit
constexpr int CP = 128 + 4;            // pitch (floats) of the output tile: conflict-free for both access patterns
constexpr int ROW_TARGET = 8;          // a scaled operand row's largest element lies in [2^8, 2^9)

// Beams per CTA (= MMA N; 8 threads each).  Key width 256 takes 64: every CTA turns the whole head's S_0 into its A
// operand, 128 KB of fp32 from L2 per tile of value rows, and at 32 beams per CTA those reads (1 GB per launch at
// 256 x 512 with 65 536 units) were what bounded the kernel; one CTA of 512 threads holds as many warps as two of 256.
template <int KD, int VD>
__host__ __device__ constexpr int tiled_beams() { return KD * VD >= 128 * 128 ? 64 : 32; }
#ifdef ONELA_TEST_HOOKS
// Test-hooks build only (a second library that the product never loads): when set, CTA (0, 0, 0) leaves out its first
// tile's MMAs and their commit, so that the wait for them runs out.
__device__ int g_hook_tiled_skip_issue;
#endif

template <int KD, int VD>
__host__ __device__ constexpr size_t tiled_smem_bytes() {
    // two A operands where there is a next tile to prepare and the key is narrow (at key width 256 the second buffer
    // leaves the fold's record loads 34 KB of L1: 89 -> 106 us at 256 x 256)
    constexpr int NB = tiled_beams<KD, VD>(), ABUF = (VD > 128 && KD <= 128) ? 2 : 1;
    return 1024 + (size_t)ABUF * (KD / 64) * 128 * 128 + (size_t)(KD / 64) * NB * 128 + (size_t)NB * CP * 4 + NB * 4 + 64;
}

// CTAs per SM the registers are capped for: small CTAs are latency-bound (a string of dependent loads per level, one MMA
// round trip), so the narrowest shape gets four.
template <int KD, int VD>
__host__ __device__ constexpr int tiled_min_ctas() { return KD + VD <= 128 ? 4 : tiled_beams<KD, VD>() == 64 ? 1 : 2; }

// DELTA: the arena keeps (alpha_t, delta_t, k_t) (Section 3.2, Eq. 2-4).  A beam owns TWO rows of the tile - its query
// and its own key, both projected through the parent state: S_{t-1} x = D S_0 x + sum_j d_j (k_j . x) delta_j, the
// replay leaving x unchanged - and after the contraction delta_t = beta_t (v_t - alpha_t S_{t-1} k_t) and
// o_t = alpha_t S_{t-1} q_t + delta_t (k_t . q_t) are formed from the two rows and the record is written; always with
// the append fused in, dk = dv <= 128.
template <int KD, int VD, typename T, typename OutT, bool DELTA = false>
__global__ void __launch_bounds__(tiled_beams<KD, VD>() * G, tiled_min_ctas<KD, VD>()) decode_tiled_kernel(const TiledArgs a) {
    constexpr int NB = tiled_beams<KD, VD>(), THREADS = NB * G;
    constexpr int BPT = DELTA ? NB / 2 : NB;          // beams per tile
    static_assert(!DELTA || (KD == VD && VD <= 128), "delta records: square heads, one tile of value rows");
    constexpr uint32_t ACC_COLS = 2 * NB;      // two accumulators of NB columns (a power of two >= 32)
    constexpr int VEC = Vec16<T>::N;
    constexpr int CK = KD / (G * VEC), CV = VD / (G * VEC);   // 16-byte chunks per lane
    static_assert(KD % 64 == 0 && VD % 64 == 0 && CK >= 1 && CV >= 1, "whole 64-element K blocks, whole chunks per lane");
    static_assert(128 % (G * VEC) == 0, "a lane's chunk lies inside one tile of 128 value rows");
    constexpr int KB = KD / 64;                   // K blocks of 64 fp16 (one 128-byte swizzled row each)
    constexpr int MT = (VD + 127) / 128;          // tiles of 128 value rows
    constexpr int A_KB = 128 * 128, R_KB = NB * 128;   // bytes of one K block of the two operands

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);      // swizzle atoms need 1024-byte alignment
    constexpr int ABUF = (MT > 1 && KD <= 128) ? 2 : 1;
    uint8_t* A_s = smem;                                               // [ABUF][KB][128 rows][128 bytes]: tile mt in buffer mt & 1
    uint8_t* R_s = A_s + ABUF * KB * A_KB;                             // [KB][NB rows][128 bytes]
    float* C_s = reinterpret_cast<float*>(R_s + KB * R_KB);            // [NB][CP]
    float* inv_s = C_s + NB * CP;                                      // [NB] what undoes a row's scales
    uint64_t* bar = reinterpret_cast<uint64_t*>(inv_s + NB);          // a tile's MMAs complete
    uint64_t* abar = bar + 1;                                          // [2] an A operand has landed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(abar + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(smem_u32(bar), 1);
        mbar_init(smem_u32(abar), 1);
        mbar_init(smem_u32(abar + 1), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ACC_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int tile = blockIdx.x, hv = blockIdx.y, req = blockIdx.z;
    const int hk = hv / a.g, Hv = a.Hk * a.g;
    const int grp = tid / G, g = tid % G;
    const int b = tile * BPT + (DELTA ? grp >> 1 : grp);
    const bool key_row = DELTA && (grp & 1);          // DELTA: the odd row of a beam projects its key
    const bool active = b < a.W;
    const int bb = active ? b : a.W - 1;  // idle units shadow a live beam so loads and shuffles stay uniform

    const float sc0 = __ldg(a.s0_scale + req * a.s0_scale_req_stride + hv);     // a power of two
    // The A operand of tile mt (S_0 rows [128 mt, 128 mt + 128), rows beyond dv zero): the store keeps every state as
    // this kernel's operand as well - fp16, times the head's scale, in 16 KB tiles of 128 rows x 64 columns laid out
    // as the MMA reads them - so a tile is dk / 64 bulk copies of 16 KB, requested by one thread, landing on a barrier
    // of their own while the CTA does something else (the fold; the previous tile's epilogue).
    const char* A_src = a.s0_f16 + req * a.s0_f16_req_stride + (long long)hv * ((long long)MT * KB * A_KB);
    int a_loads = 0, a_waits = 0;         // thread 0: A operands requested / waited for
    auto load_A = [&](int mt) {           // thread 0 only
        const uint32_t ab = smem_u32(abar + (mt & (ABUF - 1)));
        mbar_expect_tx(ab, KB * A_KB);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
            bulk_load(smem_u32(A_s + (mt & (ABUF - 1)) * (KB * A_KB) + kb * A_KB), A_src + ((long long)mt * KB + kb) * A_KB, A_KB, ab);
        ++a_loads;
    };
    // one thread: once the tile's A operand has landed, its dk / 16 MMAs into accumulator mt & 1 and the commit that
    // completes the barrier's phase (if the operand does not land in time nothing is issued, and the CTA's wait for the
    // MMAs runs out in turn)
    auto issue = [&](int mt) {
        const bool landed = mbar_wait(smem_u32(abar + (mt & (ABUF - 1))), (ABUF == 2 ? mt >> 1 : mt) & 1);
        ++a_waits;
        if (!landed) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t ad = umma_desc(smem_u32(A_s + (mt & (ABUF - 1)) * (KB * A_KB))), bd = umma_desc(smem_u32(R_s));
        constexpr uint32_t idesc = idesc_f16(NB);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                umma_f16_ss(tmem_base + (mt & 1) * NB, ad + (uint64_t)((kb * A_KB + ks * 32) >> 4),
                            bd + (uint64_t)((kb * R_KB + ks * 32) >> 4), idesc, (kb | ks) ? 1u : 0u);
        umma_commit(smem_u32(bar));
    };
    if (tid == 0) load_A(0);        // in flight while the chain is walked

    // ---- the fold (Section 3.2's recurrence applied to the query from the newest record back) ----
    const T* q = static_cast<const T*>(a.q) + (((long long)req * a.W + bb) * a.Hk + hk) * KD;
    const int32_t* table = a.table + req * a.table_req_stride;
    T* kplane = reinterpret_cast<T*>(a.kplane) + (long long)hk * a.arena_slots * a.k_stride;
    T* vplane = reinterpret_cast<T*>(a.vplane) + (long long)hv * a.arena_slots * a.v_stride;
    float2* gates = a.gates + (long long)hv * a.arena_slots;
    const bool fused = a.k_in != nullptr;      // append fused in: the newest record comes from the caller's tensors

    float r[CK * VEC], corr[CV * VEC];
#pragma unroll
    for (int c = 0; c < CK; ++c) Vec16<T>::load(q + (c * G + g) * VEC, r + c * VEC);
#pragma unroll
    for (int e = 0; e < CV * VEC; ++e) corr[e] = 0.f;
    float decay = 1.f;  // product of the alphas already passed

    // Lane g of a unit fetches the slot of the unit's ancestor at level g (the oldest eight levels: one load latency
    // for the whole chain instead of one per level); deeper levels are looked up when they are reached.
    const int old = a.depth - 1;           // records older than the beam's own: levels old - 1 .. 0
    const int32_t my_slot = g < old ? __ldg(table + (long long)g * a.max_beam + bb) : 0;
    // (two look-ups, used by two runs of the chain walk: one loop with a branch between them costs every level a
    // dozen instructions, taken or not)
    auto slot_near = [&](int level) -> int32_t { return __shfl_sync(0xffffffffu, my_slot, level, G); };          // level < G
    auto slot_far = [&](int level) -> int32_t { return __ldg(table + (long long)level * a.max_beam + bb); };    // level >= G
    struct Raw { uint4 k[CK], v[CV]; float2 gate; };          // this lane's share of a record, as stored
    auto fetch_slot = [&](long long slot) -> Raw {            // an older record, from the arena
        const uint4* kp = reinterpret_cast<const uint4*>(kplane + slot * a.k_stride) + g;
        const uint4* vp = reinterpret_cast<const uint4*>(vplane + slot * a.v_stride) + g;
        Raw x;
#pragma unroll
        for (int c = 0; c < CK; ++c) x.k[c] = __ldg(kp + c * G);
#pragma unroll
        for (int c = 0; c < CV; ++c) x.v[c] = __ldg(vp + c * G);
        x.gate = __ldg(gates + slot);
        return x;
    };
    auto fold = [&](const Raw& x) {       // c = k . r~ ;  corr += decay beta c v ;  r~ -= beta c k ;  decay *= alpha
        float kx[CK * VEC];
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            Vec16<T>::unpack(x.k[c], kx + c * VEC);
#pragma unroll
            for (int e = 0; e < VEC; ++e) dot = fmaf(kx[c * VEC + e], r[c * VEC + e], dot);
        }
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        // (DELTA, Eq. 3: the record's second half is the stored update vector, taken with the weight decay (k . x); the
        // projected vector is not changed)
        const float bc = DELTA ? dot : x.gate.y * dot;
        const float wv = decay * bc;
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            float vx[VEC];
            Vec16<T>::unpack(x.v[c], vx);
#pragma unroll
            for (int e = 0; e < VEC; ++e) corr[c * VEC + e] = fmaf(wv, vx[e], corr[c * VEC + e]);
        }
        if constexpr (!DELTA) {
#pragma unroll
            for (int e = 0; e < CK * VEC; ++e) r[e] = fmaf(-bc, kx[e], r[e]);
        }
        decay *= x.gate.x;
    };
    // The beam's own record: from its arena slot, or - append fused in - from the caller's tensors, in which case this
    // unit also writes it to the slot, bit for bit (16-byte vectors; the key once per key head, by its first value
    // head).  The fold reads the caller's copy, so nothing in this launch reads what another CTA of it writes.
    Raw cur;
    {
        const long long slot = a.bases.base[req] + bb;
        T* kdst = kplane + slot * a.k_stride;
        T* vdst = vplane + slot * a.v_stride;
        const T *ksrc = kdst, *vsrc = vdst;
        if (fused) {
            const long long krow = ((long long)req * a.W + bb) * a.Hk + hk, vrow = ((long long)req * a.W + bb) * Hv + hv;
            ksrc = static_cast<const T*>(a.k_in) + krow * KD;
            vsrc = static_cast<const T*>(a.v_in) + vrow * VD;
            cur.gate = make_float2(__ldg(a.alpha_in + vrow), __ldg(a.beta_in + vrow));
        } else {
            cur.gate = __ldg(gates + slot);
        }
#pragma unroll
        for (int c = 0; c < CK; ++c) cur.k[c] = __ldg(reinterpret_cast<const uint4*>(ksrc) + c * G + g);
#pragma unroll
        for (int c = 0; c < CV; ++c) cur.v[c] = __ldg(reinterpret_cast<const uint4*>(vsrc) + c * G + g);
        if (fused && active && !key_row) {
            if constexpr (!DELTA) {      // (the delta half of a delta record is written after the contraction)
#pragma unroll
                for (int c = 0; c < CV; ++c) reinterpret_cast<uint4*>(vdst)[c * G + g] = cur.v[c];
            }
            if (hv % a.g == 0) {
#pragma unroll
                for (int c = 0; c < CK; ++c) reinterpret_cast<uint4*>(kdst)[c * G + g] = cur.k[c];
            }
            if (g == 0) gates[slot] = cur.gate;
        }
    }
    float kq = 0.f;          // DELTA: k_t . q_t
    if constexpr (DELTA) {
        float kx[CK * VEC];
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            Vec16<T>::unpack(cur.k[c], kx + c * VEC);
#pragma unroll
            for (int e = 0; e < VEC; ++e) kq = fmaf(kx[c * VEC + e], r[c * VEC + e], kq);
        }
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) kq += __shfl_xor_sync(0xffffffffu, kq, off);
        if (key_row) {
#pragma unroll
            for (int e = 0; e < CK * VEC; ++e) r[e] = kx[e];
        }
    }
    // Narrow records are fetched one level ahead of their fold (the chain is a string of dependent loads otherwise);
    // wide ones would not fit in the registers twice.
    constexpr bool AHEAD = KD + VD <= 256;
    const int near_top = min(old, G) - 1;        // levels near_top .. 0: slots among the lanes'; old - 1 .. G: in memory
    if constexpr (DELTA) {                       // the replay runs over the older records only
        if (old > 0) {
            Raw x = old > G ? fetch_slot(slot_far(old - 1)) : fetch_slot(slot_near(old - 1));
            for (int level = old - 2; level >= G; --level) {
                const Raw next = fetch_slot(slot_far(level));
                fold(x);
                x = next;
            }
            for (int level = min(old - 2, near_top); level >= 0; --level) {
                const Raw next = fetch_slot(slot_near(level));
                fold(x);
                x = next;
            }
            fold(x);
        }
    } else if constexpr (AHEAD) {
        for (int level = old - 1; level >= G; --level) {
            const Raw next = fetch_slot(slot_far(level));
            fold(cur);
            cur = next;
        }
        for (int level = near_top; level >= 0; --level) {
            const Raw next = fetch_slot(slot_near(level));
            fold(cur);
            cur = next;
        }
        fold(cur);
    } else {
        fold(cur);
        for (int level = old - 1; level >= G; --level) {
            const Raw x = fetch_slot(slot_far(level));
            fold(x);
        }
        for (int level = near_top; level >= 0; --level) {
            const Raw x = fetch_slot(slot_near(level));
            fold(x);
        }
    }

    // ---- the folded query decay * r~ as the unit's operand row ----
    {
        float m = 0.f;
#pragma unroll
        for (int e = 0; e < CK * VEC; ++e) m = fmaxf(m, fabsf(r[e]));
#pragma unroll
        for (int off = G / 2; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        float sc, inv;
        pow2_scale(m * fabsf(decay), ROW_TARGET, sc, inv);
        const float f = decay * sc;
        if (g == 0) inv_s[grp] = inv / sc0;      // both powers of two
#pragma unroll
        for (int c = 0; c < CK; ++c) {
            const int el0 = (c * G + g) * VEC;   // first element of the chunk
            uint8_t* p = R_s + (el0 >> 6) * R_KB + grp * 128 + ((((el0 & 63) >> 3) ^ (grp & 7)) << 4) + (el0 & 7) * 2;
            const float* x = r + c * VEC;
            if constexpr (VEC == 8) {
                *reinterpret_cast<uint4*>(p) = make_uint4(pack_f16x2(x[0] * f, x[1] * f), pack_f16x2(x[2] * f, x[3] * f),
                                                          pack_f16x2(x[4] * f, x[5] * f), pack_f16x2(x[6] * f, x[7] * f));
            } else {
                *reinterpret_cast<uint2*>(p) = make_uint2(pack_f16x2(x[0] * f, x[1] * f), pack_f16x2(x[2] * f, x[3] * f));
            }
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
#ifdef ONELA_TEST_HOOKS
    if (tid == 0 && !(g_hook_tiled_skip_issue && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)) issue(0);
#else
    if (tid == 0) issue(0);
#endif

    OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + b) * Hv + hv) * VD;
    const int quad = warp & 3, half = warp >> 2;     // tensor-memory lane quadrant of this warp, and which 16 beams it takes
    bool failed = false;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        // this tile's part of corr, one row per unit
#pragma unroll
        for (int c = 0; c < CV; ++c) {
            if ((c * G * VEC) / 128 != mt) continue;
            float* dst = C_s + grp * CP + (c * G + g) * VEC - mt * 128;
#pragma unroll
            for (int e = 0; e < VEC; e += 4)
                *reinterpret_cast<float4*>(dst + e) = make_float4(corr[c * VEC + e], corr[c * VEC + e + 1], corr[c * VEC + e + 2], corr[c * VEC + e + 3]);
        }
        if (ABUF == 2 && mt + 1 < MT && tid == 0) {
            // the next tile's A operand, under this tile's MMAs: its buffer was last read by tile mt - 1, whose
            // completion this thread has waited for
            load_A(mt + 1);
        }
        const bool ok = mbar_wait(smem_u32(bar), mt & 1);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ABUF == 2) {
            // ... and its MMAs, under this tile's epilogue: their accumulator was read out before the barrier that
            // ended the previous iteration
            if (mt + 1 < MT && tid == 0) issue(mt + 1);
        } else if (mt + 1 < MT && tid == 0) {        // one A operand: free now; its MMAs go out after the barrier below
            load_A(mt + 1);
        }
        {
            uint32_t v[16];
            tmem_ld16(tmem_base + (mt & 1) * NB + half * 16 + ((uint32_t)(quad * 32) << 16), v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int i = quad * 32 + lane;          // value row within the tile
            if (mt * 128 + i < VD) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float* cell = C_s + (half * 16 + j) * CP + i;
                    *cell = fmaf(__uint_as_float(v[j]), inv_s[half * 16 + j], *cell);
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (ABUF == 1 && mt + 1 < MT && tid == 0) issue(mt + 1);
        if constexpr (DELTA) {
            // Eq. 2 and 4 on the beam's two rows (even: S_{t-1} q_t, odd: S_{t-1} k_t), by the even row's lanes:
            //   delta_t = beta_t (v_t - alpha_t S_{t-1} k_t) ,  o_t = alpha_t S_{t-1} q_t + delta_t (k_t . q_t)
            if (active && !key_row) {
                T* ddst = vplane + (long long)(a.bases.base[req] + bb) * a.v_stride;
#pragma unroll
                for (int c = 0; c < CV; ++c) {
                    const float* uq = C_s + grp * CP + (c * G + g) * VEC;
                    float vx[VEC], dl[VEC], o[VEC];
                    Vec16<T>::unpack(cur.v[c], vx);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        dl[e] = cur.gate.y * fmaf(-cur.gate.x, uq[CP + e], vx[e]);
                        o[e] = fmaf(dl[e], kq, cur.gate.x * uq[e]);
                    }
                    store_out<OutT, VEC>(out + (c * G + g) * VEC, o);
                    store_out<T, VEC>(ddst + (c * G + g) * VEC, dl);
                }
            }
        } else if (active) {
#pragma unroll
            for (int c = 0; c < CV; ++c) {
                if ((c * G * VEC) / 128 != mt) continue;
                const float* src = C_s + grp * CP + (c * G + g) * VEC - mt * 128;
                float x[VEC];
#pragma unroll
                for (int e = 0; e < VEC; e += 4) {
                    const float4 t = *reinterpret_cast<const float4*>(src + e);
                    x[e] = t.x; x[e + 1] = t.y; x[e + 2] = t.z; x[e + 3] = t.w;
                }
                store_out<OutT, VEC>(out + (c * G + g) * VEC, x);
            }
        }
        if (mt + 1 < MT) __syncthreads();      // the tile is read out before the next corr rows overwrite it
    }
    if (tid == 0) {
        // a CTA must not exit with bulk copies still landing in its shared memory: after a wait ran out nobody may
        // have waited for the A operand requested last (requests use the two barriers in turn, in order)
        for (; a_waits < a_loads; ++a_waits)
            mbar_wait(smem_u32(abar + (a_waits & (ABUF - 1))), (ABUF == 2 ? a_waits >> 1 : a_waits) & 1);
    }
    if (failed && tid == 0) {
        if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z));
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(ACC_COLS) : "memory");
    }
}

template <int KD, int VD, typename T, typename OutT, bool DELTA = false>
cudaError_t launch_one(const TiledArgs& a, cudaStream_t stream) {
    auto kern = decode_tiled_kernel<KD, VD, T, OutT, DELTA>;
    constexpr int NB = tiled_beams<KD, VD>(), THREADS = NB * G, BPT = DELTA ? NB / 2 : NB;
    constexpr size_t smem = tiled_smem_bytes<KD, VD>();
    static_assert(smem <= 232448, "shared memory per CTA");
    // One-time set-up per instantiation and device (function attributes belong to a device's context).
    constexpr int MAX_DEVICES = 64;
    static std::mutex setup_mutex;
    static bool ready[MAX_DEVICES] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(setup_mutex);
        if (!ready[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            // shared memory for the CTAs the registers allow and no more: what is left of the SM's 228 KB serves the
            // fold's record loads as L1 (asking for all of it made 128 x 128 fp32 14 % slower)
            constexpr int pct = (int)((tiled_min_ctas<KD, VD>() * (smem + 1024) * 100 + 228 * 1024 - 1) / (228 * 1024));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, pct > 100 ? 100 : pct);
            if (e != cudaSuccess) return e;
            ready[dev] = true;
        }
    }
    dim3 grid((a.W + BPT - 1) / BPT, a.Hk * a.g, a.req_count);
    kern<<<grid, THREADS, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int KD, int VD, bool DELTA = false>
cudaError_t launch_dims(const TiledArgs& a, int32_t rec_dtype, int32_t out_dtype, cudaStream_t stream) {
    if (rec_dtype == ONELA_DTYPE_BF16) {
        return out_dtype == ONELA_DTYPE_BF16 ? launch_one<KD, VD, __nv_bfloat16, __nv_bfloat16, DELTA>(a, stream)
                                             : launch_one<KD, VD, __nv_bfloat16, float, DELTA>(a, stream);
    }
    return out_dtype == ONELA_DTYPE_BF16 ? launch_one<KD, VD, float, __nv_bfloat16, DELTA>(a, stream)
                                         : launch_one<KD, VD, float, float, DELTA>(a, stream);
}

}  // namespace

#ifdef ONELA_TEST_HOOKS
extern "C" int onela_testhook_tiled_skip_issue(int on) {
    return (int)cudaMemcpyToSymbol(g_hook_tiled_skip_issue, &on, sizeof(int));
}
#endif

bool decode_tiled_supported(int32_t dk, int32_t dv) {
    return (dk == 64 && dv == 64) || (dk == 128 && (dv == 128 || dv == 256 || dv == 512)) || (dk == 256 && (dv == 256 || dv == 512));
}

cudaError_t launch_decode_tiled(const TiledArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                                cudaStream_t stream) {
    if (a.delta) {       // (alpha, delta, k) records: square heads, the append fused in
        if (!a.k_in || a.g != 1) return cudaErrorInvalidValue;
        if (dk == 64 && dv == 64) return launch_dims<64, 64, true>(a, rec_dtype, out_dtype, stream);
        if (dk == 128 && dv == 128) return launch_dims<128, 128, true>(a, rec_dtype, out_dtype, stream);
        return cudaErrorInvalidValue;
    }
    if (dk == 64 && dv == 64) return launch_dims<64, 64>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 128) return launch_dims<128, 128>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 256) return launch_dims<128, 256>(a, rec_dtype, out_dtype, stream);
    if (dk == 128 && dv == 512) return launch_dims<128, 512>(a, rec_dtype, out_dtype, stream);
    if (dk == 256 && dv == 256) return launch_dims<256, 256>(a, rec_dtype, out_dtype, stream);
    if (dk == 256 && dv == 512) return launch_dims<256, 512>(a, rec_dtype, out_dtype, stream);
    return cudaErrorInvalidValue;
}

}  // namespace onela
