// Fused decode kernel for B200 (sm_100a): dk = dv = 128, bf16 records.
//
// One persistent CTA per SM (512 threads) walks a contiguous range of work items (request, head, tile of
// TN beams).  Consecutive tiles of one (request, head) form a segment; per segment the CTA brings in,
// with bulk async copies signalled on mbarriers,
//   - the head's S_0 (the pre-swizzled TF32 image kept in the store): ONE contiguous 64 KiB copy,
//   - the DISTINCT ancestor records of the oldest chain levels (as many whole levels as fit): beams of a
//     request share ancestors, so each shared record crosses L2 -> SM once per segment instead of once
//     per beam, and the fold reads it from shared memory at shared-memory latency.
// The CTA is split into NP independent pipelines of TN*8 threads, each working on its own tiles with its
// own named barrier, operand buffers, mbarrier and tensor-memory columns, so one pipeline's waits
// (DRAM, MMA completion) are filled by the others.  Per tile a pipeline does:
//   1. fold  - a group of 8 lanes owns one (beam, head) unit and folds its query through the unit's
//              records newest -> oldest (c = k.r; corr += beta c v; r -= beta c k; decay kept as a scalar;
//              packed fp32x2 FMAs).  The beam's own record and query were prefetched during the previous
//              tile; records of levels that are not staged are gathered with coalesced 16-byte read-only
//              loads, one level ahead; staged levels come from shared memory.
//   2. meet  - the TN folded queries go to shared memory as a K-major, 128-byte-swizzled operand; one
//              thread issues 16 tcgen05.mma (kind::tf32, M = dv = 128, N = TN, K = 8), fp32 accumulation
//              in tensor memory.
//   3. finish- tcgen05.ld brings the [dv x TN] accumulator back, it is transposed through shared memory,
//              the fold groups add their corr registers and store coalesced rows.
// Every wait is bounded: on expiry the pipeline records ONELA_E_TIMEOUT in the status word and stops
// working (it still joins the CTA-wide barriers), and the CTA releases its tensor memory and returns.
#include <cstdio>

#include "onela_internal.h"
#include "onela_layout.cuh"
#include "onela_sm100.cuh"

namespace onela {

namespace {

using namespace sm100;

constexpr int OP = DV + 4;                     // pitch (floats) of the transposed accumulator
constexpr int R_TOTAL = 96 * 128 * 4;          // all pipelines' folded-query operands: up to 96 beams x 512 B
constexpr int O_TOTAL = 96 * OP * 4;           // all pipelines' output tiles (corr, then corr + accumulator)
constexpr int STAGE_CAP = 120;                 // distinct ancestor records staged per segment
constexpr int STAGE_BYTES = STAGE_CAP * REC_BYTES;
constexpr int GATE_BYTES = STAGE_CAP * 8;
constexpr int SMEM_BYTES = S0_BYTES + R_TOTAL + O_TOTAL + STAGE_BYTES + GATE_BYTES + 128 + 1024;
constexpr uint32_t TMEM_COLS = 128;            // accumulator columns: one per beam in flight
// LPU lanes per unit, PT threads per pipeline (TU = PT/LPU units folded at a time), RND rounds of units per
// tile (one MMA group per tile over N = RND * TU beams: issuing a tcgen05.mma costs ~90 cycles whatever its N,
// so tiles are wide), NP pipelines per CTA.
template <typename OutT, int LPU, int PT, int RND, int NP>
__global__ void __launch_bounds__(PT* NP, 1) decode_sm100_kernel(const DecodeArgs a, int total_tiles, int tiles_per_pair) {
    using L = Lanes<LPU>;
    using RecT = typename L::R;
    constexpr int NCH = L::NCH, NP2 = L::NP2;
    constexpr int TU = PT / LPU;          // units per round
    constexpr int N = TU * RND;           // beams per tile = MMA N
    constexpr int R_BYTES = N * 128 * 4, R_KB_STRIDE = N * 128;
    constexpr int O_FLOATS = N * OP;
    static_assert(N % 16 == 0 && N <= 256 && (R_KB_STRIDE % 1024) == 0, "MMA N and swizzle-atom alignment");
    static_assert(NP * R_BYTES <= R_TOTAL && NP * O_FLOATS * 4 <= O_TOTAL && NP * N <= (int)TMEM_COLS, "buffers");
    static_assert(PT % 128 == 0 || PT >= 128, "a pipeline needs four warps on the four tensor-memory lane quadrants");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pipe = tid / PT, ptid = tid - pipe * PT, pwarp = ptid >> 5;
    const int grp = ptid / LPU, g = ptid % LPU;

    const uint32_t s0_addr = base;
    const uint32_t r_addr = base + S0_BYTES + pipe * R_BYTES;
    uint8_t* R_s = smem + S0_BYTES + pipe * R_BYTES;
    float* O_s = reinterpret_cast<float*>(smem + S0_BYTES + R_TOTAL) + pipe * O_FLOATS;
    uint8_t* stage = smem + S0_BYTES + R_TOTAL + O_TOTAL;
    float2* gates_s = reinterpret_cast<float2*>(stage + STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(stage + STAGE_BYTES + GATE_BYTES);
    // bars[0] S_0 image, bars[1] staged records, bars[2 + p] pipeline p's MMA; then the tmem slot and the abort flag
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 + NP);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const uint32_t bar_s0 = smem_u32(bars), bar_stage = smem_u32(bars + 1), bar_mma = smem_u32(bars + 2 + pipe);
    const int bar_id = 1 + pipe;

    if (tid == 0) {
        mbar_init(bar_s0, 1);
        mbar_init(bar_stage, 32);
        for (int p = 0; p < NP; ++p) mbar_init(smem_u32(bars + 2 + p), 1);
        *abort_flag = 0;
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
    const uint32_t tmem_acc = *tmem_slot + (uint32_t)(pipe * N);   // this pipeline's accumulator columns

    // contiguous range of tiles for this CTA
    const int t_begin = (int)(((long long)blockIdx.x * total_tiles) / gridDim.x);
    const int t_end = (int)(((long long)(blockIdx.x + 1) * total_tiles) / gridDim.x);

    const char* kv = a.kv;
    const __nv_bfloat16* qbase = static_cast<const __nv_bfloat16*>(a.q);
    const int old = a.depth - 1;          // records older than a beam's own: levels old-1 .. 0
    uint32_t seg_phase = 0, mma_phase = 0;
    bool dead = false;                    // this pipeline gave up after a timeout (uniform across the pipeline)

#ifdef ONELA_TIMING
    unsigned long long gt0; unsigned smid;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt0));
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    long long tph[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long tk = clock64();
    const long long tstart = tk;
#define ONELA_TICK(i) { const long long now = clock64(); tph[i] += now - tk; tk = now; }
#else
#define ONELA_TICK(i)
#endif

    // What a unit's fold needs first: the query and the beam's own record.
    struct UnitHead {
        uint4 q[NCH];
        RecT own;
    };

    for (int seg_begin = t_begin, seg_end; seg_begin < t_end; seg_begin = seg_end) {
        const int pair = seg_begin / tiles_per_pair;
        seg_end = min(t_end, (pair + 1) * tiles_per_pair);
        const int req = pair / a.H, h = pair - req * a.H;
        const long long plane_row0 = (long long)h * a.arena_slots;
        const long long own_row0 = plane_row0 + a.bases.base[req];
        const int32_t* table_r = a.table + req * a.table_req_stride;
        const int32_t* sidx_r = a.sidx + req * a.sidx_req_stride;

        // How many of the oldest levels fit in the staging buffer (whole levels only; uniform over the CTA).
        int staged_levels = 0, n_staged = 0;
        {
            const int32_t* uoff = a.uoff + req * a.uoff_req_stride;
            for (int l = 0; l < old; ++l) {
                const int e = __ldg(uoff + l + 1);
                if (e > STAGE_CAP) break;
                staged_levels = l + 1;
                n_staged = e;
            }
        }

        // Everything of the previous segment has been consumed: each pipeline waited for its last MMA
        // (the S_0 image is free) and finished its last fold (the staged records are free).
        __syncthreads();
        if (warp == 0) {
            if (lane == 0) {
                mbar_expect_tx(bar_s0, S0_BYTES);
                bulk_load(s0_addr, a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK), S0_BYTES, bar_s0);
            }
            const int32_t* ulist = a.ulist + req * a.ulist_req_stride;
            const int mine = (n_staged > lane) ? (n_staged - lane + 31) / 32 : 0;
            mbar_expect_tx(bar_stage, mine * REC_BYTES);   // one arrival per lane, with the bytes it is about to request
            for (int i = lane; i < n_staged; i += 32) {
                const long long row = plane_row0 + __ldg(ulist + i);
                bulk_load(smem_u32(stage + i * REC_BYTES), kv + row * REC_BYTES, REC_BYTES, bar_stage);
            }
        }
        // the gates of the staged records: plain loads by every pipeline (same values), published to the
        // pipeline by the barrier each pipeline takes before its first staged read
        {
            const int32_t* ulist = a.ulist + req * a.ulist_req_stride;
            for (int i = ptid; i < n_staged; i += PT) gates_s[i] = __ldg(a.gates + plane_row0 + __ldg(ulist + i));
        }

        auto beam_of = [&](int tile, int rnd) { return (tile - pair * tiles_per_pair) * N + rnd * TU + grp; };
        auto open_unit = [&](int bb) {
            UnitHead u;
            const uint4* qp = reinterpret_cast<const uint4*>(qbase + (((long long)req * a.W + bb) * a.H + h) * DK) + g;
#pragma unroll
            for (int c = 0; c < NCH; ++c) u.q[c] = __ldg(qp + c * LPU);
            u.own = L::load_global(kv, a.gates, own_row0 + bb, g);
            return u;
        };

        // tiles go to the pipelines round-robin over the CTA's whole range, so the pipelines stay within one
        // tile of each other however the range is cut into segments
        int tile = seg_begin + (pipe - (seg_begin - t_begin) % NP + NP) % NP;
        UnitHead th;
        if (tile < seg_end && !dead) th = open_unit(min(beam_of(tile, 0), a.W - 1));
        bool first_in_seg = true;
        for (; tile < seg_end && !dead; tile += NP) {
            // Heads of the later rounds: copied asynchronously into those rounds' own, still unused, operand
            // rows (record chunks into the R row's four 128-byte pieces, query and gates into the O row).
#pragma unroll
            for (int rnd = 1; rnd < RND; ++rnd) {
                const int bb = min(beam_of(tile, rnd), a.W - 1);
                const int u = rnd * TU + grp;
                const char* rec = kv + (own_row0 + bb) * REC_BYTES;
                const char* qrow = reinterpret_cast<const char*>(qbase + (((long long)req * a.W + bb) * a.H + h) * DK);
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int ci = c * LPU + g;   // 16-byte chunk of a 256-byte vector
                    cp_async16(smem_u32(R_s + (ci >> 3) * R_KB_STRIDE + u * 128 + (ci & 7) * 16), rec + ci * 16);
                    cp_async16(smem_u32(R_s + (2 + (ci >> 3)) * R_KB_STRIDE + u * 128 + (ci & 7) * 16), rec + 256 + ci * 16);
                    cp_async16(smem_u32(O_s + u * OP) + ci * 16, qrow + ci * 16);
                }
                if (g == 0) cp_async8(smem_u32(O_s + u * OP) + 256, a.gates + own_row0 + bb);
            }
            if (RND > 1) asm volatile("cp.async.commit_group;" ::: "memory");

            // Ask L2 for the heads of this pipeline's NEXT tile now, a whole tile ahead of their loads: seven
            // 128-byte lines per unit (record 4, query 2, gates 1), one per lane.
            if (tile + NP < seg_end && g < 7) {
#pragma unroll
                for (int rnd = 0; rnd < RND; ++rnd) {
                    const int bb = min(beam_of(tile + NP, rnd), a.W - 1);
                    const char* rec = kv + (own_row0 + bb) * REC_BYTES;
                    const char* qrow = reinterpret_cast<const char*>(qbase + (((long long)req * a.W + bb) * a.H + h) * DK);
                    const char* line = g < 4 ? rec + g * 128
                                             : (g < 6 ? qrow + (g - 4) * 128 : reinterpret_cast<const char*>(a.gates + own_row0 + bb));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
                }
            }
            int failed = 0;
#pragma unroll
            for (int rnd = 0; rnd < RND; ++rnd) {
                const int bb = min(beam_of(tile, rnd), a.W - 1);   // idle groups shadow a live beam: uniform control flow
                const int u = rnd * TU + grp;                      // row of this unit in the tile's operand buffers

                // ---- 1. fold ----------------------------------------------------------------------
                // the unit's lanes keep the indices of its first levels (position in the staged list for staged
                // levels, arena slot otherwise); deeper chains read the rest on demand
                constexpr int NIDX = LPU >= 8 ? 1 : 8 / LPU;   // lanes of a unit hold the first max(LPU, 8) levels
                int32_t my_idx[NIDX];
#pragma unroll
                for (int j = 0; j < NIDX; ++j) {
                    const int lv = j * LPU + g;
                    my_idx[j] = lv < old ? __ldg((lv < staged_levels ? sidx_r : table_r) + (long long)lv * a.max_beam + bb) : 0;
                }
                auto idx_of = [&](int level) -> int32_t {
                    int32_t s = 0;
#pragma unroll
                    for (int j = 0; j < NIDX; ++j) {
                        const int32_t t = __shfl_sync(0xffffffffu, my_idx[j], level & (LPU - 1), LPU);
                        if (j == (level / LPU)) s = t;
                    }
                    return level < NIDX * LPU
                               ? s
                               : __ldg((level < staged_levels ? sidx_r : table_r) + (long long)level * a.max_beam + bb);
                };
                UnitHead uh;
                if (rnd == 0) {
                    uh = th;
                } else {
                    if (rnd == 1) {
                        asm volatile("cp.async.wait_all;" ::: "memory");
                        __syncwarp();
                    }
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int ci = c * LPU + g;
                        uh.own.k[c] = *reinterpret_cast<const uint4*>(R_s + (ci >> 3) * R_KB_STRIDE + u * 128 + (ci & 7) * 16);
                        uh.own.v[c] = *reinterpret_cast<const uint4*>(R_s + (2 + (ci >> 3)) * R_KB_STRIDE + u * 128 + (ci & 7) * 16);
                        uh.q[c] = reinterpret_cast<const uint4*>(O_s + u * OP)[ci];
                    }
                    uh.own.gate = *reinterpret_cast<const float2*>(O_s + u * OP + 64);
                    __syncwarp();   // every lane has read the scratch before any lane overwrites it below
                }

                float2 r[NP2], corr[NP2];
#ifdef ONELA_TIMING
                // make the head's arrival visible to the phase clock: touch one word of each load
                if ((uh.q[0].x ^ uh.own.k[0].x ^ uh.own.v[NCH - 1].w ^ __float_as_uint(uh.own.gate.x)) == 0x12345678u) tph[7]++;
                if (rnd == 0) ONELA_TICK(2) else ONELA_TICK(4)   // head arrival of round 0 / later rounds
#endif
#pragma unroll
                for (int c = 0; c < NCH; ++c) unpack8(uh.q[c], r + 4 * c);
#pragma unroll
                for (int e = 0; e < NP2; ++e) corr[e] = make_float2(0.f, 0.f);
                float decay = 1.f;

                // own record, then the gathered levels old-1 .. staged_levels from global memory
                L::fold_chain(uh.own, old - 1, staged_levels,
                              [&](int level) { return L::load_global(kv, a.gates, plane_row0 + idx_of(level), g); }, r, corr,
                              decay);
                if (staged_levels > 0) {
                    if (first_in_seg) {
                        // the pipeline barrier publishes the staged gates written above; the mbarrier the records
                        failed |= bar_or(bar_id, PT, 0);
                        if (!mbar_wait(bar_stage, seg_phase)) failed = 1;
                        first_in_seg = false;
                    }
                    const RecT newest = L::load_shared(stage, gates_s, idx_of(staged_levels - 1), g);
                    L::fold_chain(newest, staged_levels - 2, 0,
                                  [&](int level) { return L::load_shared(stage, gates_s, idx_of(level), g); }, r, corr, decay);
                }

                ONELA_TICK(0)   // fold arithmetic
                // ---- 2. operands: folded query -> K-major swizzled row u; corr -> row u of the output tile
                {
                    const int sw = u & 7;
                    const float2 dc = make_float2(decay, decay);
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int ci = c * LPU + g;                 // elements [8 ci, 8 ci + 8)
                        const int kb = ci >> 2;                     // K block of 32 floats
                        const int ch = 2 * (ci & 3);                // first of two 16-byte chunks inside the 128-byte row
                        uint8_t* row = R_s + kb * R_KB_STRIDE + u * 128;
                        float2 x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) x[e] = __fmul2_rn(r[4 * c + e], dc);
                        *reinterpret_cast<float4*>(row + (((ch) ^ sw) << 4)) =
                            make_float4(round_tf32(x[0].x), round_tf32(x[0].y), round_tf32(x[1].x), round_tf32(x[1].y));
                        *reinterpret_cast<float4*>(row + (((ch + 1) ^ sw) << 4)) =
                            make_float4(round_tf32(x[2].x), round_tf32(x[2].y), round_tf32(x[3].x), round_tf32(x[3].y));
                        float* orow = O_s + u * OP + ci * 8;
                        *reinterpret_cast<float4*>(orow) = make_float4(corr[4 * c].x, corr[4 * c].y, corr[4 * c + 1].x, corr[4 * c + 1].y);
                        *reinterpret_cast<float4*>(orow + 4) =
                            make_float4(corr[4 * c + 2].x, corr[4 * c + 2].y, corr[4 * c + 3].x, corr[4 * c + 3].y);
                    }
                }
            }
            ONELA_TICK(7)   // operand writes
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            failed |= *abort_flag;
            failed = bar_or(bar_id, PT, failed);
            ONELA_TICK(1)   // barrier A
            if (failed) {
                dead = true;
                break;
            }

            // The next tile's first query and record start their trip now and land during the MMA and the
            // epilogue.  (Issued after the proxy fence above: that fence waits for loads in flight.)
            if (tile + NP < seg_end) th = open_unit(min(beam_of(tile + NP, 0), a.W - 1));

            if (ptid == 0) {
                bool ok = mbar_wait(bar_s0, seg_phase);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (ok) {
                    constexpr uint32_t idesc = idesc_tf32(N);
                    const uint64_t ad = umma_desc(s0_addr), bd = umma_desc(r_addr);
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_tf32(tmem_acc, ad + (uint64_t)((kb * (DV * 128) + ks * 32) >> 4),
                                      bd + (uint64_t)((kb * R_KB_STRIDE + ks * 32) >> 4), idesc, (kb | ks) ? 1u : 0u);
                } else {
                    failed = 1;
                }
                umma_commit(bar_mma);   // arrives when the MMAs above (if any) have completed
            }
            ONELA_TICK(3)   // MMA issue (issuing thread)

            // ---- 3. finish ----------------------------------------------------------------------------
            if (!mbar_wait(bar_mma, mma_phase)) failed = 1;
            mma_phase ^= 1;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            ONELA_TICK(3)   // MMA wait (added to the issue column)
            if (pwarp < 4) {
                // the pipeline's first four warps sit on the four lane quadrants of tensor memory: each adds
                // accumulator rows (dv) 32*(warp&3) + lane of every beam of the tile onto the stored corr
                const int i = (warp & 3) * 32 + lane;
                const uint32_t taddr = tmem_acc + ((uint32_t)((warp & 3) * 32) << 16);
#pragma unroll
                for (int c0 = 0; c0 < N; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(taddr + c0, v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j) O_s[(c0 + j) * OP + i] += __uint_as_float(v[j]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            failed = bar_or(bar_id, PT, failed);
            ONELA_TICK(5)   // tmem ld + add + barrier B
            if (failed) {
                dead = true;
                break;
            }

#pragma unroll
            for (int rnd = 0; rnd < RND; ++rnd) {
                const int b = beam_of(tile, rnd);
                const int u = rnd * TU + grp;
                if (b < a.W) {
                    OutT* out = static_cast<OutT*>(a.out) + (((long long)req * a.W + b) * a.H + h) * DV;
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int e0 = (c * LPU + g) * 8;
                        const float4 x0 = *reinterpret_cast<const float4*>(O_s + u * OP + e0);
                        const float4 x1 = *reinterpret_cast<const float4*>(O_s + u * OP + e0 + 4);
                        const float o[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                        store8<OutT>(out + e0, o);
                    }
                }
            }
            ONELA_TICK(6)   // store
        }
        if (dead && ptid == 0) {
            *abort_flag = 1;
            if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)blockIdx.x;
        }
        seg_phase ^= 1;
    }
#ifdef ONELA_TIMING
    if (tid == 0 && (a.depth == 1)) {
        unsigned long long gt1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt1));
        printf("span cta %d sm %u start %llu end %llu\n", (int)blockIdx.x, smid, gt0 % 100000000ull, gt1 % 100000000ull);
    }
    if ((ptid == 0 || ptid == PT - 1) && pipe == NP - 1 && (blockIdx.x == 0 || blockIdx.x == gridDim.x / 2 || blockIdx.x == gridDim.x - 1))
        printf("cta %d tid %d depth %d tiles %d total %lld | head0 %lld headN %lld foldmath %lld opwrite %lld barA %lld mma %lld ld+barB %lld store %lld\n",
               (int)blockIdx.x, tid, a.depth, t_end - t_begin, clock64() - tstart, tph[2], tph[4], tph[0], tph[7], tph[1], tph[3], tph[5], tph[6]);
#endif

    // A CTA must not exit with bulk copies still landing in its shared memory.  In normal operation every
    // segment's copies were waited for by the threads that consumed them; after a timeout (pipelines gave
    // up early) wait for the last segment's copies here, again with a limit.
    if (tid == 0 && *abort_flag && t_begin < t_end) {
        mbar_wait(bar_s0, seg_phase ^ 1);
        mbar_wait(bar_stage, seg_phase ^ 1);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(TMEM_COLS) : "memory");
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

template <typename OutT, int LPU, int PT, int RND, int NP>
cudaError_t launch_t(const DecodeArgs& a, cudaStream_t stream) {
    auto kern = decode_sm100_kernel<OutT, LPU, PT, RND, NP>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    constexpr int N = PT / LPU * RND;
    const int tiles_per_pair = (a.W + N - 1) / N;
    const int total_tiles = a.req_count * a.H * tiles_per_pair;
    // one CTA per SM; a CTA wants at least one tile per pipeline
    const int want = (total_tiles + NP - 1) / NP;
    const int grid = want < sm_count() ? (want < 1 ? 1 : want) : sm_count();
    kern<<<grid, PT * NP, SMEM_BYTES, stream>>>(a, total_tiles, tiles_per_pair);
    return cudaGetLastError();
}

#ifndef ONELA_LPU
#define ONELA_LPU 8
#endif
#ifndef ONELA_PT
#define ONELA_PT 192
#endif
#ifndef ONELA_RND
#define ONELA_RND 2
#endif
#ifndef ONELA_PIPES
#define ONELA_PIPES 2
#endif

}  // namespace

bool decode_sm100_supported(int32_t dk, int32_t dv, int32_t rec_dtype) {
    return dk == 128 && dv == 128 && rec_dtype == ONELA_DTYPE_BF16;
}

cudaError_t launch_decode_sm100(const DecodeArgs& a, int32_t out_dtype, cudaStream_t stream) {
    return out_dtype == ONELA_DTYPE_BF16 ? launch_t<__nv_bfloat16, ONELA_LPU, ONELA_PT, ONELA_RND, ONELA_PIPES>(a, stream)
                                         : launch_t<float, ONELA_LPU, ONELA_PT, ONELA_RND, ONELA_PIPES>(a, stream);
}

}  // namespace onela
