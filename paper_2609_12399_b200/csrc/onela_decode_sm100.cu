// Warp-specialised fused decode kernel for B200 (sm_100a): dk = dv = 128, bf16 records.
//
// One persistent CTA per SM, 16 warps in two roles coupled only by mbarriers:
//   * 12 FOLD warps.  8 lanes own one (beam, head) unit; a warp folds 4 units at a time ("quad"): query
//     folded through the unit's records newest -> oldest (c = k.r; corr += beta c v; r -= beta c k; decay a
//     scalar; packed fp32x2 FMAs).  A quad's query and own record arrive through a per-warp ring of 16-byte
//     async copies, two quads ahead; with the append fused in they come from the caller's token tensors and
//     the warp also writes them to the arena.  Results go into a ring slot in shared memory: the folded query
//     as a row of the K-major 128-byte-swizzled MMA operand (rounded to TF32), corr as a row of the slot's
//     corr tile.
//   * 4 EPILOGUE warps (one per tensor-memory lane quadrant).  One lane issues the group's 16 MMAs once all
//     its rows are written; when they have completed the four warps read the accumulator, add it onto the
//     corr tile, store the outputs as coalesced 16-byte rows and hand the slot back.
// Two ring slots (operand rows, corr tile, 48 accumulator columns each) keep the MMA and the epilogue of one
// group under the folds of the next.  Work = groups of 48 consecutive beams of one (request, head), a
// contiguous range per CTA chosen on the host; consecutive groups of one head form a segment, per which all
// warps load the head's S_0 into tensor memory (rounded to TF32; it is the MMA's A operand there) and the
// epilogue warps stage the oldest chain levels in shared memory, one 512-byte bulk copy per DISTINCT
// ancestor record (as many whole levels as fit).
// The kernel is launched as a programmatic dependent launch: it sets itself up and reads the first S_0 while
// the previous kernel of the stream drains, and waits for that kernel before it touches anything else.
// Every wait is bounded and also gives up when another role has raised the abort flag; a role that gives up
// records ONELA_E_TIMEOUT, stops working but keeps joining the per-segment CTA barriers; before returning
// the CTA waits (bounded) for copies still in flight and frees its tensor memory.
#include <cstdio>

#include "onela_internal.h"
#include "onela_layout.cuh"
#include "onela_sm100.cuh"

namespace onela {

namespace {

using namespace sm100;

#ifndef ONELA_FOLD_WARPS
#define ONELA_FOLD_WARPS 12
#endif
#ifndef ONELA_LPU
#define ONELA_LPU 8
#endif
constexpr int FOLD_WARPS = ONELA_FOLD_WARPS;
constexpr int LPU = ONELA_LPU;                      // lanes per (beam, head) unit
constexpr int UPW = 32 / LPU;                       // units a fold warp folds at a time (a "quad" when LPU = 8)
constexpr int NCH = 16 / LPU;                       // 16-byte chunks per lane per 256-byte vector
constexpr int QPG = (FOLD_WARPS * UPW == 32) ? 2 : 1;   // quads each fold warp contributes to a group
constexpr int THREADS = (FOLD_WARPS + 4) * 32;      // + 4 epilogue warps (16 warps: four per SM sub-partition)
constexpr int GN = FOLD_WARPS * UPW * QPG;          // beams per group = MMA N (64 or 48)
constexpr int R_KB_STRIDE = GN * 128;               // bytes between the four 32-float K blocks of the operand
constexpr int R_BYTES = 4 * R_KB_STRIDE;            // 32768
constexpr int C_BYTES = GN * DV * 4;                // 32768: corr tile, row = beam
constexpr int SLOT_BYTES = R_BYTES + C_BYTES;
#ifndef ONELA_SLOTS
#define ONELA_SLOTS 2
#endif
constexpr int SLOTS = ONELA_SLOTS;
constexpr int HEAD_BYTES = UPW * (REC_BYTES + DK * 2);   // one quad's heads: own records + queries of its units
#ifndef ONELA_HEAD_STAGES
#define ONELA_HEAD_STAGES 1
#endif
constexpr int HEAD_STAGES = ONELA_HEAD_STAGES;          // heads in flight per fold warp
constexpr int HEADS_TOTAL = FOLD_WARPS * HEAD_STAGES * HEAD_BYTES;
#ifndef ONELA_STAGE_MAX
#define ONELA_STAGE_MAX 104
#endif
constexpr int STAGE_ROOM = (232448 - 1024 - 256 - SLOTS * SLOT_BYTES - HEADS_TOTAL) / (REC_BYTES + 8) / 4 * 4;
constexpr int STAGE_CAP = STAGE_ROOM > ONELA_STAGE_MAX ? ONELA_STAGE_MAX : STAGE_ROOM;   // distinct ancestor records staged per segment
constexpr int STAGE_BYTES = STAGE_CAP * REC_BYTES;
constexpr int GATE_BYTES = STAGE_CAP * 8;
#ifndef ONELA_SMEM_PAD
#define ONELA_SMEM_PAD 0
#endif
constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + STAGE_BYTES + GATE_BYTES + HEADS_TOTAL + 256 + 1024 + ONELA_SMEM_PAD;
constexpr uint32_t S0_COL = SLOTS * GN <= 128 ? 128 : SLOTS * GN;   // accumulators of the ring slots first, then the head's S_0
constexpr uint32_t TMEM_COLS = S0_COL + 128 <= 256 ? 256 : 512;
static_assert(S0_COL + 128 <= 512, "tensor memory columns");
static_assert(SMEM_BYTES <= 232448, "shared memory per CTA");
static_assert(HEAD_STAGES >= 1 && HEAD_STAGES <= 3, "head ring depth");
using L = Lanes<LPU>;
using RecT = L::R;

// Bounded wait that also gives up as soon as the CTA's abort flag is raised.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (int i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63 && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Position of 16-byte chunk q (4 floats) of a corr-tile row: chunks swap in pairs in every other 128-byte stretch,
// which keeps the fold warps' 32-byte-strided writes and the epilogue's 32-byte-strided reads off shared banks.
__device__ __forceinline__ int corr_chunk(int q) { return q ^ ((q >> 3) & 1); }

struct Head {           // what a unit's fold needs first
    uint4 q[NCH];
    RecT own;
};

#ifdef ONELA_TIMELINE
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ unsigned long long g_marks[64];
__device__ int g_nmarks;
#define ONELA_MARK(name) if (blockIdx.x == 0 && lane == 0) { const int mi = atomicAdd(&g_nmarks, 1); if (mi < 32) { g_marks[2 * mi] = gtime(); g_marks[2 * mi + 1] = (unsigned long long)(name[0]) | ((unsigned long long)(name[1]) << 8) | ((unsigned long long)(name[2]) << 16) | ((unsigned long long)(name[3]) << 24) | ((unsigned long long)warp << 32); } }
#else
#define ONELA_MARK(name)
#endif

#ifdef ONELA_SPAN
__device__ unsigned long long g_span[64][160][4];
__device__ __forceinline__ unsigned long long gtime2() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#endif

// Contiguous ranges of groups, one per CTA, balanced on the host with the cost of starting a segment counted in.
constexpr int MAX_CTAS = 160;
struct Partition {
    int32_t begin[MAX_CTAS + 1];
};

template <typename OutT>
__global__ void __launch_bounds__(THREADS, 1) decode_ws_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ Partition part,
                                                               int groups_per_pair, int launch_id) {
    extern __shared__ uint8_t smem_raw[];
#ifdef ONELA_SPAN
    if (threadIdx.x == 0) g_span[launch_id & 63][blockIdx.x][0] = gtime2();
#endif
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (warp == 0 || warp == FOLD_WARPS) { ONELA_MARK("start") }
    uint8_t* ring = smem;
    uint8_t* stage = ring + SLOTS * SLOT_BYTES;
    float2* gates_s = reinterpret_cast<float2*>(stage + STAGE_BYTES);
    uint8_t* heads = stage + STAGE_BYTES + GATE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(heads + HEADS_TOTAL);
    // bars: 0 S_0 in tensor memory, 1 staged records, then per ring slot s: full, MMA done, free
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 + 3 * SLOTS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const uint32_t bar_s0 = smem_u32(bars), bar_stage = smem_u32(bars + 1);
    auto bar_full = [&](int s) { return smem_u32(bars + 2 + s); };
    auto bar_done = [&](int s) { return smem_u32(bars + 2 + SLOTS + s); };
    auto bar_free = [&](int s) { return smem_u32(bars + 2 + 2 * SLOTS + s); };

    if (tid == 0) {
        mbar_init(bar_s0, THREADS / 32);              // every warp, once its share of S_0 sits in tensor memory
        mbar_init(bar_stage, 128);                    // every lane of the four epilogue warps
        for (int s = 0; s < SLOTS; ++s) {
            mbar_init(bar_full(s), QPG * FOLD_WARPS); // one arrival per quad of 4 beams
            mbar_init(bar_done(s), 1);                // tcgen05.commit
            mbar_init(bar_free(s), 4);                // the four epilogue warps
        }
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
    const uint32_t tmem_base = *tmem_slot;
    if (warp == 0) { ONELA_MARK("prologue done") }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next launch may set itself up under this one

    const int g_begin = part.begin[blockIdx.x], g_end = part.begin[blockIdx.x + 1];
    const int old = a.depth - 1;          // records older than a beam's own: levels old-1 .. 0
    const bool fused = a.k_in != nullptr;  // append fused in: the newest record comes from the caller's tensors
    const char* kv = a.kv;
    const __nv_bfloat16* qbase = static_cast<const __nv_bfloat16*>(a.q);

#ifdef ONELA_TIMING
    long long tph[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long t_issue = 0;
    long long tk = clock64();
    const long long tstart = tk;
#define ONELA_TICK(i) { const long long now = clock64(); tph[i] += now - tk; tk = now; }
#else
#define ONELA_TICK(i)
#endif
    bool dead = false;                    // this warp gave up (timeout or abort raised elsewhere)
    int heads_issued = 0, heads_taken = 0;   // fold warps: quads whose heads were requested / consumed so far
    const int grp = lane / LPU, g = lane % LPU;

    // S_0 of a (request, head) goes to tensor memory, rounded to TF32 on the way: it is the MMA's A operand there, so
    // there is no shared-memory copy of S_0 and no S_0 traffic per MMA.  Row-major fp32 in the store; lane i of
    // tensor memory holds row i.  Every warp takes the 32 rows of its lane quadrant and one block of 32 columns,
    // so the whole 64 KiB costs one load latency; the next segment's S_0 is requested into L2 on the way.
    auto load_s0 = [&](int pair_now, bool has_next) {
        const int quad = warp & 3, i = quad * 32 + lane;
        const int req = pair_now / a.H, h = pair_now - req * a.H;
        const float* row = a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK) + (long long)i * DK;
#pragma unroll 1
        for (int kb = warp >> 2; kb < 4; kb += THREADS / 128) {
            uint32_t v[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 x = __ldg(reinterpret_cast<const float4*>(row + kb * 32) + c);
                v[4 * c] = __float_as_uint(round_tf32(x.x)); v[4 * c + 1] = __float_as_uint(round_tf32(x.y));
                v[4 * c + 2] = __float_as_uint(round_tf32(x.z)); v[4 * c + 3] = __float_as_uint(round_tf32(x.w));
            }
            tmem_st32(tmem_base + S0_COL + kb * 32 + ((uint32_t)(quad * 32) << 16), v);
            if (has_next) {
                const int nreq = (pair_now + 1) / a.H, nh = (pair_now + 1) - nreq * a.H;
                const float* nrow = a.s0 + nreq * a.s0_req_stride + (long long)nh * (DV * DK) + (long long)i * DK + kb * 32;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nrow));
            }
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_s0);
    };
    // The first segment's S_0 is read before the launch's dependencies are waited for: the store is written only
    // by the state calls (a copy or a prefill kernel), and a reorder launch always separates those from a decode.
    if (g_begin < g_end) {
        const int pair0 = g_begin / groups_per_pair;
        load_s0(pair0, (pair0 + 1) * groups_per_pair < g_end);
    }
    // Everything below reads what earlier launches of the stream wrote (tokens, queries, ancestry rows).
    asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef ONELA_SPAN
    if (threadIdx.x == 0) g_span[launch_id & 63][blockIdx.x][2] = gtime2();
#endif

    int seg_idx = 0;
    for (int sg_begin = g_begin, sg_end; sg_begin < g_end; sg_begin = sg_end, ++seg_idx) {
        const int pair = sg_begin / groups_per_pair;
        sg_end = min(g_end, (pair + 1) * groups_per_pair);
        const int req = pair / a.H, h = pair - req * a.H;
        const long long plane_row0 = (long long)h * a.arena_slots;
        const long long own_row0 = plane_row0 + a.bases.base[req];
        const uint32_t seg_parity = seg_idx & 1;
        const int gcount0 = sg_begin - g_begin;   // groups this CTA finished before this segment

        // ---- fold warps: head prefetch machinery.  Quad k of the segment: group sg_begin + k / QPG.
        const int n_quads = QPG * (sg_end - sg_begin);
        auto group_of = [&](int k) { return QPG == 2 ? (k >> 1) : k; };
        auto half_of = [&](int k) { return QPG == 2 ? (k & 1) : 0; };
        auto beam_of = [&](int k) { return ((sg_begin + group_of(k)) - pair * groups_per_pair) * GN + half_of(k) * (FOLD_WARPS * UPW) + UPW * warp + grp; };
        // The heads of a quad (own record and query of its four units) arrive by 16-byte async copies into a
        // two-stage ring private to the warp, two quads ahead of their use (each lane copies exactly the
        // chunks it reads back); the gates ride in registers.
        auto slot_of = [&](int k) { return (gcount0 + group_of(k)) % SLOTS; };
        auto use_of = [&](int k) { return (gcount0 + group_of(k)) / SLOTS; };
        auto row_of = [&](int k) { return half_of(k) * (FOLD_WARPS * UPW) + UPW * warp + grp; };
        uint8_t* my_heads = heads + (warp < FOLD_WARPS ? warp : 0) * (HEAD_STAGES * HEAD_BYTES);
        auto q_row = [&](int bb) { return reinterpret_cast<const char*>(qbase + (((long long)req * a.W + bb) * a.H + h) * DK); };
        auto issue_head = [&](int k) {   // every lane copies the chunks it will read back itself
            const int st = heads_issued % HEAD_STAGES;
            const int bb = min(beam_of(k), a.W - 1);             // idle units shadow a live beam
            const uint32_t dst = smem_u32(my_heads + st * HEAD_BYTES);
            const char* qr = q_row(bb) + g * 16;
            if (fused) {   // the call's records come straight from the caller's k and v tensors
                const long long in_row = ((long long)req * a.W + bb) * a.H + h;
                const char* kr = static_cast<const char*>(a.k_in) + in_row * (DK * 2) + g * 16;
                const char* vr = static_cast<const char*>(a.v_in) + in_row * (DV * 2) + g * 16;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    cp_async16(dst + grp * REC_BYTES + (c * LPU + g) * 16, kr + c * LPU * 16);
                    cp_async16(dst + grp * REC_BYTES + (16 + c * LPU + g) * 16, vr + c * LPU * 16);
                }
            } else {
                const char* rec = kv + (own_row0 + bb) * REC_BYTES + g * 16;
#pragma unroll
                for (int c = 0; c < 2 * NCH; ++c) cp_async16(dst + grp * REC_BYTES + (c * LPU + g) * 16, rec + c * LPU * 16);
            }
#pragma unroll
            for (int c = 0; c < NCH; ++c) cp_async16(dst + UPW * REC_BYTES + grp * (DK * 2) + (c * LPU + g) * 16, qr + c * LPU * 16);
            asm volatile("cp.async.commit_group;" ::: "memory");
#ifdef ONELA_TIMING
            t_issue = clock64();
#endif
            ++heads_issued;
#ifndef ONELA_L2_AHEAD
#define ONELA_L2_AHEAD 1
#endif
#if ONELA_L2_AHEAD > 0
            // the quad after this one: its 128-byte lines are requested into L2 (no shared memory needed for them yet)
            if (k + ONELA_L2_AHEAD < n_quads && lane < UPW * 6) {
                const int un = lane / 6, item = lane % 6;
                const int b2 = min(beam_of(k + ONELA_L2_AHEAD) - grp + un, a.W - 1);
                const long long in_row = ((long long)req * a.W + b2) * a.H + h;
                const char* base_p = item < 2 ? reinterpret_cast<const char*>(qbase) + in_row * (DK * 2)
                                   : fused ? (item < 4 ? static_cast<const char*>(a.k_in) + in_row * (DK * 2)
                                                       : static_cast<const char*>(a.v_in) + in_row * (DV * 2))
                                           : kv + (own_row0 + b2) * REC_BYTES + (item < 4 ? 0 : 256);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(base_p + (item & 1) * 128));
            }
#endif
        };
        auto load_gate = [&](int k) {
            const int bb = min(beam_of(k), a.W - 1);
            if (!fused) return __ldg(a.gates + own_row0 + bb);
            const long long in_row = ((long long)req * a.W + bb) * a.H + h;
            return make_float2(__ldg(a.alpha_in + in_row), __ldg(a.beta_in + in_row));
        };
        // The segment's first heads go out before anything else: they depend on nothing the segment sets up.
        float2 gate0 = make_float2(1.f, 0.f), gate1 = gate0;
        if (warp < FOLD_WARPS && !dead && n_quads > 0) {
            issue_head(0);
            gate0 = load_gate(0);
            if (1 < n_quads) gate1 = load_gate(1);
#pragma unroll
            for (int st = 1; st < HEAD_STAGES; ++st)
                if (st < n_quads) issue_head(st);
        }

        // How many of the oldest levels fit in the staging buffer (whole levels only; uniform over the CTA).
        // Lane l looks at level l (one load latency for the whole chain); offsets grow with the level.
        int staged_levels = 0, n_staged = 0;
        {
            const int32_t* uoff = a.uoff + req * a.uoff_req_stride;
            const int e = (lane < old) ? __ldg(uoff + lane + 1) : 0x7fffffff;
            staged_levels = __popc(__ballot_sync(0xffffffffu, e <= STAGE_CAP));
            n_staged = __shfl_sync(0xffffffffu, e, staged_levels > 0 ? staged_levels - 1 : 0);
            if (staged_levels == 0) n_staged = 0;
        }

        // The previous segment is fully consumed: the epilogue warps pass this barrier only after the last
        // group's MMA completed and was read back; the fold warps after their last staged read.
        __syncthreads();
        if (warp >= FOLD_WARPS && warp < FOLD_WARPS + 4 && !dead) {
            // The epilogue warps (idle until the first group is folded) stage the distinct records: one 512-byte bulk
            // copy per record, its gates by a plain load, one record per lane.  Every lane arrives once, announcing
            // the bytes it requested; its gate store is ordered before the arrival.
            static_assert(STAGE_CAP <= 128, "one staged record per epilogue lane");
            const int i = (warp - FOLD_WARPS) * 32 + lane;
            if (i < n_staged) {
                const long long row = plane_row0 + __ldg(a.ulist + req * a.ulist_req_stride + i);
                bulk_load(smem_u32(stage + i * REC_BYTES), kv + row * REC_BYTES, REC_BYTES, bar_stage);
                gates_s[i] = __ldg(a.gates + row);
            }
            mbar_expect_tx(bar_stage, i < n_staged ? REC_BYTES : 0);
        }
        if (seg_idx > 0 && !dead) load_s0(pair, sg_end < g_end);

        // One thread issues a group's 16 MMAs as soon as all its rows are written (never a fold warp: whichever fold
        // warp issued would be the last to finish its next quad).  Returns true when it had to give up.
        auto issue_group = [&](int s, int use) -> bool {
            int mma_failed = 0;
            if (lane == 0) {
                bool ok = wait_or_abort(bar_full(s), use & 1, abort_flag);
                ok = ok && wait_or_abort(bar_s0, seg_parity, abort_flag);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                ONELA_TICK(0)   // (issuer) wait for the group's rows
                if (ok) {
                    constexpr uint32_t idesc = idesc_tf32(GN);
                    const uint64_t bd = umma_desc(smem_u32(ring + s * SLOT_BYTES));
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_tf32_ts(tmem_base + s * GN, tmem_base + S0_COL + (kb * 4 + ks) * 8,
                                         bd + (uint64_t)((kb * R_KB_STRIDE + ks * 32) >> 4), idesc, (kb | ks) ? 1u : 0u);
                } else {
                    mma_failed = 1;
                }
                umma_commit(bar_done(s));   // arrives when the MMAs above (if any) have completed
                ONELA_TICK(1)   // (issuer) issue
                ONELA_MARK("mma issued")
            }
            return __shfl_sync(0xffffffffu, mma_failed, 0) != 0;
        };

        if (warp < FOLD_WARPS) {
            // =============================== FOLD ===============================
            const int32_t* table_r = a.table + req * a.table_req_stride;
            const int32_t* sidx_r = a.sidx + req * a.sidx_req_stride;
            constexpr int NIDX = LPU >= 8 ? 1 : 8 / LPU;     // the unit's lanes hold the indices of its first 8 levels
            struct Idx { int32_t v[NIDX]; };
            auto load_idx = [&](int k) -> Idx {
                const int bb = min(beam_of(k), a.W - 1);
                Idx x;
#pragma unroll
                for (int j = 0; j < NIDX; ++j) {
                    const int lv = j * LPU + g;
                    x.v[j] = lv < old ? __ldg((lv < staged_levels ? sidx_r : table_r) + (long long)lv * a.max_beam + bb) : 0;
                }
                return x;
            };
            Idx idx_next{};
            if (!dead && n_quads > 0) idx_next = load_idx(0);
            bool staged_ready = false;
            for (int k = 0; k < n_quads && !dead; ++k) {
                const int s = slot_of(k), use = use_of(k);
                const int u = row_of(k);                         // row of this unit in the slot
                const int bb = min(beam_of(k), a.W - 1);
                Head cur;
                {
                    const int st = heads_taken % HEAD_STAGES;
                    // the oldest copy group in flight is this quad's; a newer one (the next quad's) may stay pending
                    const int newer = heads_issued - heads_taken - 1;
                    if (newer >= 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
                    else if (newer == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
                    else asm volatile("cp.async.wait_group 0;" ::: "memory");
                    ONELA_TICK(5)   // (fold warps) wait for the head
#ifdef ONELA_TIMING
                    tph[4] += clock64() - t_issue;   // issue -> arrival observed (one stage in flight)
#endif
                    if (warp == 0) { ONELA_MARK("head arrived") }
                    const uint4* rec = reinterpret_cast<const uint4*>(my_heads + st * HEAD_BYTES + grp * REC_BYTES) + g;
                    const uint4* qv = reinterpret_cast<const uint4*>(my_heads + st * HEAD_BYTES + UPW * REC_BYTES + grp * (DK * 2)) + g;
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        cur.own.k[c] = rec[c * LPU];
                        cur.own.v[c] = rec[16 + c * LPU];
                        cur.q[c] = qv[c * LPU];
                    }
                    cur.own.gate = gate0;
                    ++heads_taken;
                    if (fused && beam_of(k) < a.W) {   // the append: this beam's record goes to its arena slot, bit for bit
                        uint4* dst = reinterpret_cast<uint4*>(a.kv_out + (own_row0 + bb) * REC_BYTES) + g;
#pragma unroll
                        for (int c = 0; c < NCH; ++c) {
                            dst[c * LPU] = cur.own.k[c];
                            dst[16 + c * LPU] = cur.own.v[c];
                        }
                        if (g == 0) a.gates_out[own_row0 + bb] = gate0;
                    }
                }
                gate0 = gate1;
#ifdef ONELA_TIMING
                if ((cur.q[0].x ^ cur.own.k[0].x ^ cur.own.v[NCH - 1].w) == 0x12345678u) tph[7]++;
                ONELA_TICK(6)   // (fold warps) read the head from the stage
#endif
                if (k + HEAD_STAGES < n_quads) issue_head(k + HEAD_STAGES);
                if (k + 2 < n_quads) gate1 = load_gate(k + 2);
                ONELA_TICK(2)   // (fold warps) issue the head after next

                // lane g keeps the index of level g (position in the staged list for staged levels, arena slot
                // otherwise); it was fetched while the previous quad was folded, the next quad's is fetched now
                const Idx my_idx = idx_next;
                if (k + 1 < n_quads) idx_next = load_idx(k + 1);
                auto idx_of = [&](int level) -> int32_t {
                    int32_t t = 0;
#pragma unroll
                    for (int j = 0; j < NIDX; ++j) {
                        const int32_t x = __shfl_sync(0xffffffffu, my_idx.v[j], level & (LPU - 1), LPU);
                        if (j == level / LPU) t = x;
                    }
                    return level < NIDX * LPU ? t
                                              : __ldg((level < staged_levels ? sidx_r : table_r) + (long long)level * a.max_beam + bb);
                };

#ifdef ONELA_TIMING
                if ((cur.q[0].x ^ cur.own.k[0].x ^ cur.own.v[NCH - 1].w ^ __float_as_uint(cur.own.gate.x)) == 0x12345678u) tph[7]++;
                ONELA_TICK(0)   // head arrival (+ issue of next head)
#endif
                float2 r[4 * NCH], corr[4 * NCH];
#pragma unroll
                for (int c = 0; c < NCH; ++c) unpack8(cur.q[c], r + 4 * c);
#pragma unroll
                for (int e = 0; e < 4 * NCH; ++e) corr[e] = make_float2(0.f, 0.f);
                float decay = 1.f;
                L::fold_chain_simple(cur.own, old - 1, staged_levels,
                              [&](int level) { return L::load_global(kv, a.gates, plane_row0 + idx_of(level), g); }, r, corr, decay);
                if (staged_levels > 0) {
                    if (!staged_ready) {
                        if (!wait_or_abort(bar_stage, seg_parity, abort_flag)) { dead = true; break; }
                        staged_ready = true;
                    }
                    const RecT newest = L::load_shared(stage, gates_s, idx_of(staged_levels - 1), g);
                    L::fold_chain_simple(newest, staged_levels - 2, 0,
                                  [&](int level) { return L::load_shared(stage, gates_s, idx_of(level), g); }, r, corr, decay);
                }

                ONELA_TICK(1)   // fold
                // the slot must have been handed back by the epilogue of its previous use
                if (use > 0 && !wait_or_abort(bar_free(s), (use - 1) & 1, abort_flag)) { dead = true; break; }
                ONELA_TICK(7)   // wait for the slot
                uint8_t* R_s = ring + s * SLOT_BYTES;
                float* C_s = reinterpret_cast<float*>(R_s + R_BYTES);
                {
                    // Bank conflicts: the lanes g and g + 4 of a unit own the same chunk positions of two operand rows
                    // 48 * 128 bytes apart, so the upper four lanes write their two chunks in the opposite order;
                    // the corr tile (a layout of our own) swaps each pair of 16-byte chunks in every other 128-byte
                    // stretch of a row instead (corr_chunk below; the epilogue reads it the same way).
                    const int sw = u & 7;
                    const bool hi = (g >> 2) & 1;
                    const float2 dc = make_float2(decay, decay);
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int ci = c * LPU + g;                 // elements [8 ci, 8 ci + 8)
                        const int kb = ci >> 2, ch = 2 * (ci & 3);  // K block of 32 floats; first of two 16-byte chunks
                        uint8_t* row = R_s + kb * R_KB_STRIDE + u * 128;
                        float2 x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) x[e] = __fmul2_rn(r[4 * c + e], dc);
                        const float4 lo4 = make_float4(round_tf32(x[0].x), round_tf32(x[0].y), round_tf32(x[1].x), round_tf32(x[1].y));
                        const float4 hi4 = make_float4(round_tf32(x[2].x), round_tf32(x[2].y), round_tf32(x[3].x), round_tf32(x[3].y));
                        *reinterpret_cast<float4*>(row + (((ch + (hi ? 1 : 0)) ^ sw) << 4)) = hi ? hi4 : lo4;
                        *reinterpret_cast<float4*>(row + (((ch + (hi ? 0 : 1)) ^ sw) << 4)) = hi ? lo4 : hi4;
                        float* crow = C_s + u * DV;
                        *reinterpret_cast<float4*>(crow + corr_chunk(2 * ci) * 4) =
                            make_float4(corr[4 * c].x, corr[4 * c].y, corr[4 * c + 1].x, corr[4 * c + 1].y);
                        *reinterpret_cast<float4*>(crow + corr_chunk(2 * ci + 1) * 4) =
                            make_float4(corr[4 * c + 2].x, corr[4 * c + 2].y, corr[4 * c + 3].x, corr[4 * c + 3].y);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
                __syncwarp();
                ONELA_TICK(3)   // operand write + proxy fence
                if (warp == 0) { ONELA_MARK("quad written") }
                if (lane == 0) mbar_arrive(bar_full(s));
                ONELA_TICK(4)   // arrive
            }
        } else {
            // =============================== EPILOGUE ===============================
            const int quad = warp & 3;                    // tensor-memory lane quadrant of this warp
            const int i = quad * 32 + lane;               // output element (dv index) of this thread
            for (int gi = sg_begin; gi < sg_end && !dead; ++gi) {
                const int gcount = gcount0 + (gi - sg_begin);
                const int s = gcount % SLOTS, use = gcount / SLOTS;
                if (warp == FOLD_WARPS && issue_group(s, use)) { dead = true; break; }
                if (!wait_or_abort(bar_done(s), use & 1, abort_flag)) { dead = true; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                ONELA_TICK(5)   // epilogue: wait for the MMA group
                if (warp == FOLD_WARPS) { ONELA_MARK("mma done") }
                float* C_s = reinterpret_cast<float*>(ring + s * SLOT_BYTES + R_BYTES);
                const int b0 = (gi - pair * groups_per_pair) * GN;
                const uint32_t taddr = tmem_base + s * GN + ((uint32_t)(quad * 32) << 16);
                {
                    // accumulator rows (dv) of this thread, all 64 beams, added onto the corr tile in place
                    uint32_t v[GN];
                    if (GN == 64) {
                        tmem_ld64(taddr, v);
                    } else {
#pragma unroll
                        for (int c0 = 0; c0 < GN; c0 += 16) tmem_ld16(taddr + c0, v + c0);
                    }
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int ip = corr_chunk(i >> 2) * 4 + (i & 3);   // where the corr tile keeps element i of a row
#pragma unroll
                    for (int j = 0; j < GN; ++j) C_s[j * DV + ip] += __uint_as_float(v[j]);
                }
                ONELA_TICK(2)   // tmem ld + add
                if (bar_or(1, 128, 0)) { dead = true; break; }     // the four epilogue warps: tile complete
                {
                    // coalesced stores: 16 lanes cover one beam's 128 outputs, 8 elements each
                    const int et = (warp - FOLD_WARPS) * 32 + lane;
#pragma unroll
                    for (int it = 0; it < GN * 16 / 128; ++it) {   // GN * 16 chunks of 16 bytes over 128 threads
                        const int idx = it * 128 + et, j = idx >> 4, ch = idx & 15;
                        if (b0 + j < a.W) {
                            const float4 x0 = *reinterpret_cast<const float4*>(C_s + j * DV + corr_chunk(2 * ch) * 4);
                            const float4 x1 = *reinterpret_cast<const float4*>(C_s + j * DV + corr_chunk(2 * ch + 1) * 4);
                            const float o[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                            store8<OutT>(static_cast<OutT*>(a.out) + (((long long)req * a.W + b0 + j) * a.H + h) * DV + ch * 8, o);
                        }
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free(s));
                ONELA_TICK(6)   // epilogue: read back, add, store
                if (warp == FOLD_WARPS) { ONELA_MARK("epilogue done") }
            }
        }
        if (dead) {
            if (lane == 0) {
                *abort_flag = 1;
                if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)blockIdx.x;
            }
        }
    }

#ifdef ONELA_TIMING
    if (lane == 0 && (warp == 0 || warp == 5 || warp == FOLD_WARPS || warp == FOLD_WARPS + 1) && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1) && (a.depth == 1 || a.depth == 8))
        printf("cta %d warp %d depth %d groups %d total %lld | head %lld fold %lld slotwait %lld write %lld arrive+mma %lld | t5 %lld t2 %lld t6 %lld\n",
               (int)blockIdx.x, warp, a.depth, g_end - g_begin, clock64() - tstart, tph[0], tph[1], tph[7], tph[3], tph[4], tph[5], tph[2], tph[6]);
#endif
    // A CTA must not exit with bulk copies still landing in its shared memory: after an abort nobody may
    // have waited for the last segment's copies, nor a fold warp for the heads it had requested.
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    if (tid == 0 && *abort_flag && g_begin < g_end) mbar_wait(bar_stage, (seg_idx - 1) & 1);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) { ONELA_MARK("exit") }
#ifdef ONELA_TIMELINE
    if (blockIdx.x == 0 && tid == 0) {
        const int n = min(g_nmarks, 32);
        for (int i = 0; i < n; ++i) {
            const unsigned long long tag = g_marks[2 * i + 1];
            printf("mark %c%c%c%c warp %2d t=%llu ns\n", (char)(tag & 255), (char)((tag >> 8) & 255), (char)((tag >> 16) & 255),
                   (char)((tag >> 24) & 255), (int)(tag >> 32), g_marks[2 * i] - g_marks[0]);
        }
        g_nmarks = 0;
    }
#endif
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
#ifdef ONELA_SPAN
    if (threadIdx.x == 0) g_span[launch_id & 63][blockIdx.x][1] = gtime2();
#endif
}

int sm_count_ws() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// Contiguous group ranges for the CTAs.  Starting a segment (a new (request, head): pipeline drained, S_0 reloaded,
// staging refilled) costs about as much as SEG_COST / GROUP_COST groups, so a CTA's cost is counted as
// GROUP_COST * groups + SEG_COST * segments and the smallest bound T is searched for which a greedy fill needs no
// more CTAs than there are SMs.  Returns the number of CTAs used.
#ifndef ONELA_SEG_COST
#define ONELA_SEG_COST 7
#endif
constexpr int GROUP_COST = 4, SEG_COST = ONELA_SEG_COST;
int greedy_fill(int total_groups, int gpp, int limit, int max_ctas, int32_t* begin) {
    int n = 0, gi = 0;
    while (gi < total_groups) {
        if (n == max_ctas) return max_ctas + 1;
        if (begin) begin[n] = gi;
        int cost = 0;
        bool any = false;
        while (gi < total_groups) {
            const int pair_end = (gi / gpp + 1) * gpp;
            const int room = (limit - cost - SEG_COST) / GROUP_COST;     // groups of this segment that still fit
            if (room <= 0) break;
            const int take = room < pair_end - gi ? room : pair_end - gi;
            gi += take;
            cost += SEG_COST + take * GROUP_COST;
            any = true;
            if (gi < pair_end) break;
        }
        if (!any) return max_ctas + 1;   // the bound does not admit a single group
        ++n;
    }
    if (begin) begin[n] = total_groups;
    return n;
}
int make_partition(int total_groups, int gpp, int sms, Partition* part) {
    int lo = SEG_COST + GROUP_COST, hi = SEG_COST * (total_groups / gpp + 2) + GROUP_COST * total_groups;
    while (lo < hi) {
        const int mid = (lo + hi) / 2;
        if (greedy_fill(total_groups, gpp, mid, sms, nullptr) <= sms) hi = mid;
        else lo = mid + 1;
    }
    return greedy_fill(total_groups, gpp, lo, sms, part->begin);
}

template <typename OutT>
cudaError_t launch_ws_t(const DecodeArgs& a, cudaStream_t stream) {
    auto kern = decode_ws_kernel<OutT>;
    static bool configured = false;
    static int sms = 148;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        sms = sm_count_ws();
        if (sms > MAX_CTAS) sms = MAX_CTAS;
        configured = true;
    }
    const int groups_per_pair = (a.W + GN - 1) / GN;
    const int total_groups = a.req_count * a.H * groups_per_pair;
    static thread_local Partition part;          // the last launch's partition, reused while the shape stays
    static thread_local int part_total = -1, part_gpp = -1, part_sms = -1, part_ctas = 0;
    if (part_total != total_groups || part_gpp != groups_per_pair || part_sms != sms) {
        part_ctas = make_partition(total_groups, groups_per_pair, sms, &part);
        part_total = total_groups; part_gpp = groups_per_pair; part_sms = sms;
    }
    static int launch_id = 0;
    // Programmatic dependent launch: this launch's CTAs may start, allocate and read S_0 while the previous
    // kernel of the stream drains; the kernel waits for that kernel's completion before it reads anything else.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(part_ctas);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a, part, groups_per_pair, launch_id++);
}

}  // namespace

#ifdef ONELA_SPAN
extern "C" int onela_debug_spans(unsigned long long* host_out) {   // instrumented builds only
    return (int)cudaMemcpyFromSymbol(host_out, g_span, sizeof(g_span));
}
#endif

bool decode_sm100_supported(int32_t dk, int32_t dv, int32_t rec_dtype) {
    return dk == 128 && dv == 128 && rec_dtype == ONELA_DTYPE_BF16;
}

cudaError_t launch_decode_sm100_ws(const DecodeArgs& a, int32_t out_dtype, cudaStream_t stream) {
    return out_dtype == ONELA_DTYPE_BF16 ? launch_ws_t<__nv_bfloat16>(a, stream) : launch_ws_t<float>(a, stream);
}

}  // namespace onela
