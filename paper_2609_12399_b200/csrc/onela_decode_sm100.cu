// Warp-specialised fused decode kernel for B200 (sm_100a): dk = dv = 128, bf16 records.
//
// One persistent CTA per SM, 16 warps in two roles coupled only by mbarriers:
//   * 12 FOLD warps.  8 lanes own one (beam, head) unit; a warp folds 4 units at a time ("quad"): query
//     folded through the unit's records newest -> oldest (c = k.r; corr += beta c v; r -= beta c k; decay a
//     scalar; packed fp32x2 FMAs).  A quad's query and own record arrive through a per-warp stage of 16-byte
//     async copies, one quad ahead; with the append fused in they come from the caller's token tensors and the
//     warp also writes them to the arena.  Results go into a
//     ring slot in shared memory: the folded query as a row of the K-major 128-byte-swizzled MMA operand
//     (fp16, times a power of two that keeps the row inside fp16's range), corr as a row of the slot's corr tile.
//   * 4 EPILOGUE warps (one per tensor-memory lane quadrant).  One lane of the first issues a group's 8 MMAs
//     once all its rows are written - one group ahead of the epilogue, so neither the issuing nor the MMAs'
//     latency lies between two epilogues.  When a group's MMAs have completed the four warps read the
//     accumulator and transpose it, by plain stores, over the slot's operand rows (dead by then); the other
//     three warps add that tile to the corr tile and store the outputs as coalesced 16-byte rows while the
//     first issues the next group; then the slot is handed back.  They also prepare the next segment (below)
//     while the fold warps work on the current one.
// Two ring slots (operand rows, corr tile, 48 accumulator columns each) keep the MMA and the epilogue of one
// group under the folds of the next.  Work = groups of 48 consecutive beams of one (request, head), a
// contiguous range per CTA chosen on the host; consecutive groups of one head form a segment.  Per segment the
// head's S_0 sits in tensor memory (as fp16, scaled by the head's power of two; it is the MMA's A operand there)
// and the oldest chain levels are staged in shared memory, one 512-byte bulk copy per DISTINCT ancestor record (as
// many whole levels as fit).  S_0 and the staging area are double-buffered, so a CTA moves from one segment to the next without
// draining: nothing in the main loop is a CTA-wide barrier.
// A second instantiation (GROUPED) serves grouped value heads: segments are (request, VALUE head), the query and the
// keys are those of key head h / g, and a record's two halves live in two planes (keys per key head, values per value
// head), so staging and gathers read both and the fused append writes a key once, by its first value head.
// The kernel is launched as a programmatic dependent launch: it sets itself up and reads the first S_0 while
// the previous kernel of the stream drains, and waits for that kernel before it touches anything else.
// Every wait is bounded and also gives up when another role has raised the abort flag; a role that gives up
// records ONELA_E_TIMEOUT and stops working; before returning the CTA waits (bounded) for copies still in
// flight and frees its tensor memory.
#include <cstdio>
#include <mutex>
#include <type_traits>

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
constexpr int THREADS = (FOLD_WARPS + 4) * 32;      // + 4 epilogue warps (16 warps: four per SM sub-partition)
constexpr int GN = FOLD_WARPS * UPW;                // beams per group = MMA N (48)
constexpr int R_KB_STRIDE = GN * 128;               // bytes between the two K blocks (64 fp16 each) of the operand
constexpr int R_BYTES = 4 * R_KB_STRIDE;            // a slot's first tile: the group's operand rows (its first half),
                                                    // later the transposed accumulators (all of it)
constexpr int C_BYTES = GN * DV * 4;                // corr tile, row = beam
constexpr int SLOT_BYTES = R_BYTES + C_BYTES;
constexpr int SLOTS = 2;
constexpr int HEAD_BYTES = UPW * (REC_BYTES + DK * 2);   // one quad's heads: own records + queries of its units
constexpr int HEADS_TOTAL = FOLD_WARPS * HEAD_BYTES;     // one stage per fold warp (a deeper ring measured slower)
#ifndef ONELA_STAGE_BUF
#define ONELA_STAGE_BUF 58
#endif
// Two staging buffers of STAGE_BUF distinct ancestor records each (segment s uses buffer s & 1); a CTA whose whole
// range is one segment uses them as one.  Sized so that the CTA stays within the 196 KiB shared-memory carve-out
// (what is left of the SM's 256 KiB serves the gathered records as L1).
constexpr int STAGE_BUF = ONELA_STAGE_BUF;
constexpr int STAGE_BYTES = 2 * STAGE_BUF * REC_BYTES;
constexpr int GATE_BYTES = (2 * STAGE_BUF * 8 + 127) & ~127;   // padded: the heads' stages behind it stay 128-byte aligned (measured: 1.5 % faster)
constexpr int INV_BYTES = SLOTS * GN * 4;        // per ring slot and beam: what undoes the operands' scales
#ifdef ONELA_WS_TL
constexpr int TL_EXTRA = 3 * 200 * 8;
#else
constexpr int TL_EXTRA = 0;
#endif
constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + STAGE_BYTES + GATE_BYTES + HEADS_TOTAL + 256 + INV_BYTES + 1024 + TL_EXTRA;
// DELTA instantiation (records (alpha, delta, k), forward projection replay): a beam owns TWO rows of a group - its
// query and its own key, both projected through the parent state - so a group holds GN / 2 beams; per ring slot the
// beams' own value rows (raw) and three scalars each (alpha_t, beta_t, k_t . q_t) wait for the epilogue.
constexpr int DELTA_BEAMS = GN / 2;
constexpr int DELTA_SLOT_BYTES = DELTA_BEAMS * (DV * 2) + DELTA_BEAMS * 16;
constexpr int SMEM_BYTES_DELTA = SMEM_BYTES + SLOTS * DELTA_SLOT_BYTES;
static_assert(SMEM_BYTES_DELTA <= 232448, "shared memory per CTA (delta records)");
static_assert((DELTA_BEAMS * 16) % 96 == 0, "three storing warps share a delta group's 16-byte chunks evenly");
constexpr uint32_t S0_COL = 128;                 // accumulators of the ring slots in [0, SLOTS * GN); S_0 buffers (64 columns) at 128 and 256
constexpr int R_TARGET = 8;                      // a scaled operand row's largest element lies in [2^8, 2^9) x (decay in [1, 2)): far inside fp16's range
constexpr uint32_t TMEM_COLS = 512;
static_assert(SLOTS * GN <= 128, "accumulator columns");
static_assert(R_BYTES >= C_BYTES, "the accumulators are transposed over the operand rows");
static_assert(2 * STAGE_BUF <= 128, "one staged record per epilogue lane");
static_assert(SMEM_BYTES <= 232448, "shared memory per CTA");
static_assert(GN % 16 == 0 && GN >= 16 && GN <= 256, "MMA N");
static_assert((GN * 16) % 96 == 0, "three storing warps share a group's 16-byte chunks evenly");
using L = Lanes<LPU>;
using RecT = L::R;

#ifdef ONELA_WS_TL
// Debug builds only (the timeline library; never compiled into the product): clock stamps of CTA 0's role milestones,
// kept in shared memory and written out when the CTA ends.  Roles: fold warp 0, the issuing epilogue warp, a storing one.
constexpr int TL_CAP = 200;
__device__ unsigned long long g_ws_tl[3 * TL_CAP];
__device__ int g_ws_tl_n[3];
__device__ int g_ws_tl_cta;                       // the CTA whose roles are stamped
#define TL(ev, g)                                                                                         \
    do {                                                                                                  \
        if (lane == 0 && tl_role >= 0 && tl_n < TL_CAP)                                                   \
            tl_s[tl_role * TL_CAP + tl_n++] = ((unsigned long long)(ev) << 56) | ((unsigned long long)((g) & 0xff) << 48) | \
                                              ((unsigned long long)clock64() & 0xffffffffffffull);         \
    } while (0)
constexpr int TL_BYTES = 3 * TL_CAP * 8;
#else
#define TL(ev, g) do { } while (0)
constexpr int TL_BYTES = 0;
#endif

#ifdef ONELA_TEST_HOOKS
// Test-hooks build only (a second library that the product never loads): when set, the first fold warp of CTA 0
// leaves out ONE arrival (its first quad's), so that the wait for that group's rows runs out.
__device__ int g_hook_drop_full_arrival;
#endif

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


// Contiguous ranges of groups, one per CTA, balanced on the host with the cost of starting a segment counted in.
constexpr int MAX_CTAS = DECODE_MAX_CTAS;
using Partition = DecodePartition;

// GROUPED: value head h reads the queries and keys of key head h / g; a.H counts VALUE heads, the record's k lives in
// the key heads' plane (a.kv) and its v in the value heads' plane (a.vv), 256 bytes each.
// DELTA: the arena keeps (alpha_t, delta_t, k_t) (Section 3.2, Eq. 2-4); both projections S q_t and S k_t of the parent
// state are replayed forward from S_0 . q_t and S_0 . k_t (one MMA set over the 2 x 24 rows of a group), delta_t and
// o_t are formed in the epilogue and the record is written there; always with the append fused in, never GROUPED.
template <typename OutT, bool GROUPED, bool FUSED, bool DELTA = false>
__global__ void __launch_bounds__(THREADS, 1) decode_ws_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ Partition part,
                                                               int groups_per_pair) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* ring = smem;
    uint8_t* stage = ring + SLOTS * SLOT_BYTES;
    float2* gates_s = reinterpret_cast<float2*>(stage + STAGE_BYTES);
    uint8_t* heads = stage + STAGE_BYTES + GATE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(heads + HEADS_TOTAL);
    // bars: per S_0 / staging buffer b: S_0 in tensor memory, records staged, staging buffer read out;
    //       per ring slot s: full, MMA done, free
    const uint32_t bar_s0_first = smem_u32(bars + 6 + 3 * SLOTS);   // the first segment's S_0, put there by all warps
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7 + 3 * SLOTS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* inv_s = reinterpret_cast<float*>(heads + HEADS_TOTAL + 256);      // [SLOTS][GN]
    uint8_t* delta_s = heads + HEADS_TOTAL + 256 + INV_BYTES;                // DELTA: [SLOTS][value rows | scalars]
#ifdef ONELA_WS_TL
    unsigned long long* tl_s = reinterpret_cast<unsigned long long*>(delta_s + (DELTA ? SLOTS * DELTA_SLOT_BYTES : 0));
    const int tl_role = (int)blockIdx.x != g_ws_tl_cta ? -1 : warp == 0 ? 0 : warp == FOLD_WARPS ? 1 : warp == FOLD_WARPS + 1 ? 2 : -1;
    int tl_n = 0;
#endif
    constexpr int BPG = DELTA ? DELTA_BEAMS : GN;                            // beams per group
    static_assert(!DELTA || (FUSED && !GROUPED), "delta records come with the append fused in, ungrouped");
    auto bar_s0 = [&](int b) { return smem_u32(bars + b); };
    auto bar_stage = [&](int b) { return smem_u32(bars + 2 + b); };
    auto bar_sfree = [&](int b) { return smem_u32(bars + 4 + b); };
    auto bar_full = [&](int s) { return smem_u32(bars + 6 + s); };
    auto bar_done = [&](int s) { return smem_u32(bars + 6 + SLOTS + s); };
    auto bar_free = [&](int s) { return smem_u32(bars + 6 + 2 * SLOTS + s); };

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_s0(b), 4);                  // the four epilogue warps, once S_0 sits in tensor memory
            mbar_init(bar_stage(b), 128);             // every lane of the four epilogue warps (+ the bytes they request)
            mbar_init(bar_sfree(b), FOLD_WARPS);      // every fold warp, after its last read of the buffer in a segment
        }
        for (int s = 0; s < SLOTS; ++s) {
            mbar_init(bar_full(s), FOLD_WARPS);       // one arrival per quad
            mbar_init(bar_done(s), 1);                // tcgen05.commit
            mbar_init(bar_free(s), 4);                // the four epilogue warps
        }
        mbar_init(bar_s0_first, 16);                  // the sixteen warps that bring the first S_0 in
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
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next launch may set itself up under this one
    TL(1, 0);   // tensor memory allocated, barriers ready

    const int g_begin = part.begin[blockIdx.x], g_end = part.begin[blockIdx.x + 1];
    const int pair_begin = g_begin / groups_per_pair;
    const int n_segs = g_begin < g_end ? (g_end - 1) / groups_per_pair - pair_begin + 1 : 0;
    const bool single = n_segs == 1;                       // one segment: the two staging buffers serve as one
    const int stage_cap = single ? 2 * STAGE_BUF : STAGE_BUF;
    const int old = a.depth - 1;          // records older than a beam's own: levels old-1 .. 0
    constexpr bool fused = FUSED;          // append fused in: the newest record comes from the caller's tensors
    const char* kv = a.kv;
    const __nv_bfloat16* qbase = static_cast<const __nv_bfloat16*>(a.q);
    // rows of the caller's tensors: q and k have one row per KEY head, v, the gates and the outputs per VALUE head
    // GROUPED also serves value widths of 256 and 512: a value head is cut into a.tiles value heads of 128 outputs
    // ("tiles") that share its gates and its S_0 scale; value_head(h) is the head a tile belongs to.
    auto key_head = [&](int h) { return GROUPED ? h / a.g : h; };
    auto value_head = [&](int h) { return GROUPED ? h / a.tiles : h; };
    auto krow_in = [&](int req, int bb, int h) { return ((long long)req * a.W + bb) * (GROUPED ? a.Hk : a.H) + key_head(h); };
    auto vrow_in = [&](int req, int bb, int h) { return ((long long)req * a.W + bb) * a.H + h; };
    // rows of the arena: ungrouped one 512-byte row (k | v) per (head, slot); grouped a 256-byte row in each plane
    auto k_at = [&](int h, long long slot) {
        return GROUPED ? kv + ((long long)key_head(h) * a.arena_slots + slot) * a.k_stride : kv + ((long long)h * a.arena_slots + slot) * REC_BYTES;
    };
    auto v_at = [&](int h, long long slot) {
        return GROUPED ? a.vv + ((long long)value_head(h) * a.arena_slots + slot) * a.v_stride + (h - value_head(h) * a.tiles) * (DV * 2)
                       : kv + ((long long)h * a.arena_slots + slot) * REC_BYTES + DK * 2;
    };
    const int grp = lane / LPU, g = lane % LPU;
    bool dead = false;                    // this warp gave up (timeout or abort raised elsewhere)

    // S_0 of a (request, head) goes to tensor memory as fp16 (TF32's mantissa; K = 16 per MMA instead of 8), times
    // the head's power-of-two scale from the store, which keeps it inside fp16's range whatever the caller's units:
    // it is the MMA's A operand there, so there is no shared-memory copy of S_0 and no S_0 traffic per MMA.
    // Row-major fp32 in the store; lane i of tensor memory holds row i, two elements per column; the 64 columns of
    // buffer `buf` start at S0_COL + 128 buf.  A warp takes the 32 rows of its lane quadrant and the 32-element blocks
    // kb0, kb0 + step, ...; the S_0 after this one is requested into L2 on the way.
    auto load_s0 = [&](int pair_now, int buf, int kb0, int step, bool has_next) {
        const int quad = warp & 3, i = quad * 32 + lane;
        const int req = pair_now / a.H, h = pair_now - req * a.H;
        const float* row = a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK) + (long long)i * DK;
        const float sc = __ldg(a.s0_scale + req * a.s0_scale_req_stride + value_head(h));
#pragma unroll 1
        for (int kb = kb0; kb < 4; kb += step) {
            uint32_t v[16];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 x = __ldg(reinterpret_cast<const float4*>(row + kb * 32) + c);
                v[2 * c] = pack_f16x2(x.x * sc, x.y * sc);
                v[2 * c + 1] = pack_f16x2(x.z * sc, x.w * sc);
            }
            tmem_st16(tmem_base + S0_COL + buf * 128 + kb * 16 + ((uint32_t)(quad * 32) << 16), v);
            if (has_next) {
                const int nreq = (pair_now + 1) / a.H, nh = (pair_now + 1) - nreq * a.H;
                const float* nrow = a.s0 + nreq * a.s0_req_stride + (long long)nh * (DV * DK) + (long long)i * DK + kb * 32;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nrow));
            }
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    };
    // The first segment's S_0 is requested by all warps (one 32-column block each) before the launch's dependencies are
    // waited for, and put into tensor memory after the first heads have been requested: the store is written only by
    // the state calls (a copy or a prefill kernel), and a reorder launch always separates those from a decode.
    static_assert(THREADS >= 512, "the first sixteen warps take one 32-column block of the first S_0 each");
    const bool s0_mine = warp < 16;
    float4 s0_first[8];
    float s0_first_scale = 1.f;
    if (n_segs > 0 && s0_mine) {
        const int req = pair_begin / a.H, h = pair_begin - req * a.H;
        s0_first_scale = __ldg(a.s0_scale + req * a.s0_scale_req_stride + value_head(h));
        const float* row = a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK) + (long long)((warp & 3) * 32 + lane) * DK + (warp >> 2) * 32;
#pragma unroll
        for (int c = 0; c < 8; ++c) s0_first[c] = __ldg(reinterpret_cast<const float4*>(row) + c);
        if (n_segs > 1) {
            const int nreq = (pair_begin + 1) / a.H, nh = (pair_begin + 1) - nreq * a.H;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(a.s0 + nreq * a.s0_req_stride + (long long)nh * (DV * DK) +
                                                          (long long)((warp & 3) * 32 + lane) * DK + (warp >> 2) * 32));
        }
    }
    auto put_first_s0 = [&]() {
        if (n_segs == 0 || !s0_mine) return;
        const float sc = s0_first_scale;
        uint32_t v[16];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            v[2 * c] = pack_f16x2(s0_first[c].x * sc, s0_first[c].y * sc);
            v[2 * c + 1] = pack_f16x2(s0_first[c].z * sc, s0_first[c].w * sc);
        }
        tmem_st16(tmem_base + S0_COL + (warp >> 2) * 16 + ((uint32_t)((warp & 3) * 32) << 16), v);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_s0_first);
    };
    // Each role waits for the launch's dependencies below (`dependency_wait`), before it reads anything earlier
    // launches of the stream wrote (tokens, queries, ancestry rows).  Requests of lines into L2 are not reads in that
    // sense - L2 is the point of coherence - and are made before it.
    auto dependency_wait = [&]() {
        asm volatile("griddepcontrol.wait;" ::: "memory");
    };

    // How many of the oldest levels of a request's chains fit in `stage_cap` staged records (whole levels only), and
    // how many records that is.  Lane l looks at level l (one load latency for the whole chain); warp-uniform.
    // `sparse` (optional): bit l set when level l has more than W / 4 distinct records, i.e. little sharing - the
    // levels whose gathered records are worth requesting ahead.
    auto staging_of = [&](int req, int& levels, int& count, uint32_t* sparse = nullptr) {
        const int32_t* uoff = a.uoff + req * a.uoff_req_stride;
        // (at most the eight oldest levels, whose list positions a unit's lanes hold: the staged fold then never has to
        // look an index up in memory)
        const int e_all = (lane < old) ? __ldg(uoff + lane + 1) : 0x7fffffff;
        const int e = lane < 8 ? e_all : 0x7fffffff;
        levels = __popc(__ballot_sync(0xffffffffu, e <= stage_cap));
        count = __shfl_sync(0xffffffffu, e, levels > 0 ? levels - 1 : 0);
        if (levels == 0) count = 0;
        if (sparse) {
            int prev = __shfl_up_sync(0xffffffffu, e_all, 1);
            if (lane == 0) prev = 0;
            *sparse = __ballot_sync(0xffffffffu, lane < old && (e_all - prev) * 4 > a.W);
        }
    };

    if (warp < FOLD_WARPS) {
        // =============================== FOLD ===============================
        // Quad k of this warp belongs to group g_begin + k: rows UPW * warp .. + UPW - 1 of the group.
        const int n_quads = g_end - g_begin;
        uint8_t* my_heads = heads + warp * HEAD_BYTES;
        struct Unit { int seg, req, h, gip; };           // segment, request, head, group within the (request, head) pair
        auto beam_of = [&](const Unit& u) { return u.gip * BPG + (DELTA ? (UPW * warp + grp) >> 1 : UPW * warp + grp); };
        auto live_beam = [&](const Unit& u) { return min(beam_of(u), a.W - 1); };   // idle units shadow a live beam
        auto next_unit = [&](Unit u) {                   // the quad after u's, without divisions
            if (++u.gip == groups_per_pair) {
                u.gip = 0;
                ++u.seg;
                if (++u.h == a.H) { u.h = 0; ++u.req; }
            }
            return u;
        };
        Unit u0;                                         // this warp's current quad; u1, u2: the next two
        {
            const int pair = g_begin / groups_per_pair;
            u0.seg = 0;
            u0.req = pair / a.H;
            u0.h = pair - u0.req * a.H;
            u0.gip = g_begin - pair * groups_per_pair;
        }
        // The heads of a quad (own record and query of its units) arrive by 16-byte async copies into the warp's
        // stage, one quad ahead of their use (each lane copies exactly the chunks it reads back); the gates ride in
        // registers.  The lines of the FIRST quad are requested into L2 before the launch's dependencies are waited
        // for (requesting every later quad's lines a quad ahead of its copies as well measured 2 % slower).
        auto request_heads = [&](const Unit& n) {        // the 128-byte lines of a quad's heads, into L2
            if (lane < UPW * 6) {
                const int un = lane / 6, item = lane % 6;
                const int b2 = min(n.gip * BPG + (DELTA ? (UPW * warp + un) >> 1 : UPW * warp + un), a.W - 1);
                const long long krow2 = krow_in(n.req, b2, n.h), vrow2 = vrow_in(n.req, b2, n.h);
                const long long slot2 = a.bases.base[n.req] + b2;
                const char* p2 = item < 2 ? reinterpret_cast<const char*>(qbase) + krow2 * (DK * 2)
                                 : fused  ? (item < 4 ? static_cast<const char*>(a.k_in) + krow2 * (DK * 2)
                                                      : static_cast<const char*>(a.v_in) + vrow2 * (DV * 2))
                                          : (item < 4 ? k_at(n.h, slot2) : v_at(n.h, slot2));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p2 + (item & 1) * 128));
            }
        };
        auto issue_head = [&](const Unit& u) {
            const uint32_t dst = smem_u32(my_heads);
            const int bb = live_beam(u);
            const long long krow = krow_in(u.req, bb, u.h);
            const char* qr = reinterpret_cast<const char*>(qbase + krow * DK) + g * 16;
            if (fused) {   // the call's records come straight from the caller's k and v tensors
                const char* kr = static_cast<const char*>(a.k_in) + krow * (DK * 2) + g * 16;
                const char* vr = static_cast<const char*>(a.v_in) + vrow_in(u.req, bb, u.h) * (DV * 2) + g * 16;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    cp_async16(dst + grp * REC_BYTES + (c * LPU + g) * 16, kr + c * LPU * 16);
                    cp_async16(dst + grp * REC_BYTES + (16 + c * LPU + g) * 16, vr + c * LPU * 16);
                }
            } else {
                const long long slot = a.bases.base[u.req] + bb;
                const char* kr = k_at(u.h, slot) + g * 16;
                const char* vr = v_at(u.h, slot) + g * 16;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    cp_async16(dst + grp * REC_BYTES + (c * LPU + g) * 16, kr + c * LPU * 16);
                    cp_async16(dst + grp * REC_BYTES + (16 + c * LPU + g) * 16, vr + c * LPU * 16);
                }
            }
#pragma unroll
            for (int c = 0; c < NCH; ++c) cp_async16(dst + UPW * REC_BYTES + grp * (DK * 2) + (c * LPU + g) * 16, qr + c * LPU * 16);
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        auto load_gate = [&](const Unit& u) {
            const int bb = live_beam(u);
            if (!fused) return __ldg(a.gates + (long long)value_head(u.h) * a.arena_slots + a.bases.base[u.req] + bb);
            const long long in_row = GROUPED ? ((long long)u.req * a.W + bb) * (a.H / a.tiles) + value_head(u.h) : vrow_in(u.req, bb, u.h);
            return make_float2(__ldg(a.alpha_in + in_row), __ldg(a.beta_in + in_row));
        };
        // staging layout of the request whose quads are being looked at (the same for all heads of a request)
        int info_req = -1, info_levels = 0, info_count = 0;
        uint32_t info_sparse = 0;
        auto staged_levels_of = [&](int req) {
            if (req != info_req) { staging_of(req, info_levels, info_count, &info_sparse); info_req = req; }
            return info_levels;
        };
        constexpr int NIDX = LPU >= 8 ? 1 : 8 / LPU;     // the unit's lanes hold the indices of its first 8 levels
        static_assert(NIDX * LPU >= 8, "staging_of stages up to eight levels: their indices must be among the lanes'");
        struct Idx { int32_t v[NIDX]; };
        auto load_idx = [&](const Unit& u) -> Idx {
            const int sl = staged_levels_of(u.req);
            const int bb = live_beam(u);
            const int32_t* table_r = a.table + u.req * a.table_req_stride;
            const int32_t* sidx_r = a.sidx + u.req * a.sidx_req_stride;
            Idx x;
#pragma unroll
            for (int j = 0; j < NIDX; ++j) {
                const int lv = j * LPU + g;
                x.v[j] = lv < old ? __ldg((lv < sl ? sidx_r : table_r) + (long long)lv * a.max_beam + bb) : 0;
            }
            return x;
        };

        float2 gate0 = make_float2(1.f, 0.f), gate1 = gate0;
        Idx idx_next{};
        Unit u1 = next_unit(u0), u2 = next_unit(u1);
        if (n_quads > 0) request_heads(u0);
        dependency_wait();
        if (n_quads > 0) {
            issue_head(u0);
            gate0 = load_gate(u0);
            if (1 < n_quads) gate1 = load_gate(u1);
            idx_next = load_idx(u0);
        }
        TL(2, 0);   // dependencies waited for, first heads requested
        put_first_s0();
        TL(3, 0);   // first S_0 in tensor memory
        int cur_seg = -1, buf = 0, staged_levels = 0, n_ahead = 0;
        float seg_inv_s0 = 1.f;
        bool staged_ready = false;
        long long plane_row0 = 0, own_row0 = 0;
        const int32_t *table_r = nullptr, *sidx_r = nullptr;
        // The loop exists twice, with and without the requests ahead of the gathered records (at its end): where
        // they are not wanted the loop is exactly the one without them (their mere presence measured 0.7 % slower).
        auto fold_quads = [&](auto ahead_tag) {
            constexpr bool AHEAD = decltype(ahead_tag)::value;
            for (int k = 0; k < n_quads && !dead; ++k, u0 = u1, u1 = u2, u2 = next_unit(u2)) {
                if (u0.seg != cur_seg) {          // entering a segment: nothing to wait for here
                    cur_seg = u0.seg;
                    buf = single ? 0 : (cur_seg & 1);
                    staged_ready = false;
                    staged_levels = staged_levels_of(u0.req);
                    // levels gathered from global memory whose lines are worth requesting ahead (end of the loop)
                    if (AHEAD) n_ahead = (info_sparse >> staged_levels) ? min(old - staged_levels, NIDX * LPU - staged_levels) : 0;
                    seg_inv_s0 = 1.f / __ldg(a.s0_scale + u0.req * a.s0_scale_req_stride + value_head(u0.h));   // a power of two
                    plane_row0 = (long long)value_head(u0.h) * a.arena_slots;      // row 0 of the head's gate plane
                    own_row0 = plane_row0 + a.bases.base[u0.req];
                    table_r = a.table + u0.req * a.table_req_stride;
                    sidx_r = a.sidx + u0.req * a.sidx_req_stride;
                }
                const bool seg_last = (k + 1 == n_quads) || (u1.seg != cur_seg);
                const int s = k % SLOTS, use = k / SLOTS;
                const int u = UPW * warp + grp;                  // row of this unit in the slot
                const int bb = live_beam(u0);
                Head cur;
                {
                    TL(10, k);  // fold: quad start
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    TL(11, k);  // fold: heads landed
                    const uint4* rec = reinterpret_cast<const uint4*>(my_heads + grp * REC_BYTES) + g;
                    const uint4* qv = reinterpret_cast<const uint4*>(my_heads + UPW * REC_BYTES + grp * (DK * 2)) + g;
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        cur.own.k[c] = rec[c * LPU];
                        cur.own.v[c] = rec[16 + c * LPU];
                        cur.q[c] = qv[c * LPU];
                    }
                    cur.own.gate = gate0;
                    // the next quad's copies go out before this quad's stores (each lane overwrites only the chunks it
                    // has just read)
                    if (k + 1 < n_quads) issue_head(u1);
                    if (DELTA) {
                        // the key half of the record and the gates; delta_t follows from the epilogue
                        if ((grp & 1) == 0 && beam_of(u0) < a.W) {
                            uint4* dst = reinterpret_cast<uint4*>(a.kv_out + (own_row0 + bb) * REC_BYTES) + g;
#pragma unroll
                            for (int c = 0; c < NCH; ++c) dst[c * LPU] = cur.own.k[c];
                            if (g == 0) a.gates_out[own_row0 + bb] = gate0;
                        }
                    } else if (fused && beam_of(u0) < a.W) {   // the append: this beam's record goes to its arena slot, bit for bit
                        if constexpr (GROUPED) {
                            const long long slot = a.bases.base[u0.req] + bb;
                            uint4* vdst = reinterpret_cast<uint4*>(a.vv_out + (v_at(u0.h, slot) - a.vv)) + g;
#pragma unroll
                            for (int c = 0; c < NCH; ++c) vdst[c * LPU] = cur.own.v[c];
                            if (u0.h % a.g == 0) {     // the key is stored once per key head: by its first value head
                                uint4* kdst = reinterpret_cast<uint4*>(a.kv_out + (k_at(u0.h, slot) - kv)) + g;
#pragma unroll
                                for (int c = 0; c < NCH; ++c) kdst[c * LPU] = cur.own.k[c];
                            }
                        } else {
                            uint4* dst = reinterpret_cast<uint4*>(a.kv_out + (own_row0 + bb) * REC_BYTES) + g;
#pragma unroll
                            for (int c = 0; c < NCH; ++c) {
                                dst[c * LPU] = cur.own.k[c];
                                dst[16 + c * LPU] = cur.own.v[c];
                            }
                        }
                        if (g == 0 && (!GROUPED || u0.h % a.tiles == 0)) a.gates_out[own_row0 + bb] = gate0;
                    }
                }
                gate0 = gate1;
                if (k + 2 < n_quads) gate1 = load_gate(u2);

                // lane g keeps the index of level g (position in the staged list for staged levels, arena slot
                // otherwise); it was fetched while the previous quad was folded, the next quad's is fetched now
                const Idx my_idx = idx_next;
                if (k + 1 < n_quads) idx_next = load_idx(u1);
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
                // The same for a staged level: always among the lanes' (staging_of stages no level beyond them), so no
                // branch to the look-up in memory stands in the staged fold - merely being there, never taken, it cost
                // every level a dozen instructions (2.77 -> 2.5 us per level on the beam-512 stack).
                auto staged_idx_of = [&](int level) -> int32_t {
                    if constexpr (NIDX == 1) return __shfl_sync(0xffffffffu, my_idx.v[0], level, LPU);   // level < LPU
                    int32_t t = 0;
#pragma unroll
                    for (int j = 0; j < NIDX; ++j) {
                        const int32_t x = __shfl_sync(0xffffffffu, my_idx.v[j], level & (LPU - 1), LPU);
                        if (j == level / LPU) t = x;
                    }
                    return t;
                };

                float2 r[4 * NCH], corr[4 * NCH];
                float kq = 0.f;              // DELTA: k_t . q_t
                if (DELTA) {
                    float2 kx[4 * NCH];
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        unpack8(cur.q[c], r + 4 * c);
                        unpack8(cur.own.k[c], kx + 4 * c);
                    }
                    float2 d2 = make_float2(0.f, 0.f);
#pragma unroll
                    for (int e = 0; e < 4 * NCH; ++e) d2 = __ffma2_rn(kx[e], r[e], d2);
                    kq = d2.x + d2.y;
#pragma unroll
                    for (int o = LPU / 2; o > 0; o >>= 1) kq += __shfl_xor_sync(0xffffffffu, kq, o);
                    if (grp & 1) {           // the odd unit of a beam projects its key
#pragma unroll
                        for (int e = 0; e < 4 * NCH; ++e) r[e] = kx[e];
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < NCH; ++c) unpack8(cur.q[c], r + 4 * c);
                }
#pragma unroll
                for (int e = 0; e < 4 * NCH; ++e) corr[e] = make_float2(0.f, 0.f);
                float decay = 1.f;
                // A first guess at the scale of the unit's operand row, from the query's norm and off the end-of-quad
                // path (one shuffle reduction): with keys of norm <= 1 and beta in [0, 2] a fold step never lengthens r~,
                // so |r~| stays below 2^hq, the power of two above |q|, and the guess stands.  Whether it does is checked
                // on the folded row itself (below).
                float q_scale = 1.f, q_inv = 1.f;
                {
                    float2 n2 = make_float2(0.f, 0.f);
#pragma unroll
                    for (int e = 0; e < 4 * NCH; ++e) n2 = __ffma2_rn(r[e], r[e], n2);
                    float norm2 = n2.x + n2.y;
#pragma unroll
                    for (int o = LPU / 2; o > 0; o >>= 1) norm2 += __shfl_xor_sync(0xffffffffu, norm2, o);
                    const int eb = (int)(__float_as_uint(norm2) >> 23) & 255;      // |q|^2 in [2^(eb-127), 2^(eb-126))
                    const int hq = (eb - 127 + 2) >> 1;                             // |q| < 2^hq
                    if (eb > 0 && eb < 255 && hq > -100 && hq < 100) {
                        q_scale = __uint_as_float((uint32_t)(127 + R_TARGET - hq) << 23);
                        q_inv = __uint_as_float((uint32_t)(127 + hq - R_TARGET) << 23);
                    }
                }
                auto gather = [&](int level) {
                                  const long long slot = idx_of(level);
                                  if constexpr (GROUPED) {
                                      RecT rec;
                                      const uint4* kp = reinterpret_cast<const uint4*>(k_at(u0.h, slot)) + g;
                                      const uint4* vp = reinterpret_cast<const uint4*>(v_at(u0.h, slot)) + g;
#pragma unroll
                                      for (int c = 0; c < NCH; ++c) {
                                          rec.k[c] = __ldg(kp + c * LPU);
                                          rec.v[c] = __ldg(vp + c * LPU);
                                      }
                                      rec.gate = __ldg(a.gates + plane_row0 + slot);
                                      return rec;
                                  } else {
                                      return L::load_global(kv, a.gates, plane_row0 + slot, g);
                                  }
                              };
                if (DELTA) {     // the replay runs over the older records only; the beam's own is formed in the epilogue
                    if (old - 1 >= staged_levels) {
                        const RecT first = gather(old - 1);
                        L::template fold_chain_simple<true>(first, old - 2, staged_levels, gather, r, corr, decay);
                    }
                } else {
                    L::fold_chain_simple(cur.own, old - 1, staged_levels, gather, r, corr, decay);
                }
                // The segment's staging is waited for even when it holds nothing: it keeps this warp from running past
                // the epilogue warps' preparation of the segment after next (whose barriers share these phases).
                if (!staged_ready && (staged_levels > 0 || seg_last)) {
                    if (!wait_or_abort(bar_stage(buf), (single ? 0 : (cur_seg >> 1)) & 1, abort_flag)) { dead = true; break; }
                    staged_ready = true;
                }
                if (staged_levels > 0) {
                    const uint8_t* st = stage + buf * (STAGE_BUF * REC_BYTES);
                    const float2* gs = gates_s + buf * STAGE_BUF;
                    const RecT newest = L::load_shared(st, gs, staged_idx_of(staged_levels - 1), g);
                    L::template fold_chain_simple<DELTA>(newest, staged_levels - 2, 0,
                                  [&](int level) { return L::load_shared(st, gs, staged_idx_of(level), g); }, r, corr, decay);
                }
                if (seg_last) {                    // this warp's last read of the segment's staging buffer
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_sfree(buf));
                }

                // the slot must have been handed back by the epilogue of its previous use
                TL(12, k);  // fold: folded
                if (use > 0 && !wait_or_abort(bar_free(s), (use - 1) & 1, abort_flag)) { dead = true; break; }
                TL(13, k);  // fold: slot free
                uint8_t* R_s = ring + s * SLOT_BYTES;
                float* C_s = reinterpret_cast<float*>(R_s + R_BYTES);
                {
                    // Bank conflicts: the lanes g and g + 4 of a unit own the same chunk positions of two operand rows
                    // 48 * 128 bytes apart, so the upper four lanes write their two chunks in the opposite order;
                    // the corr tile (a layout of our own) swaps each pair of 16-byte chunks in every other 128-byte
                    // stretch of a row instead (corr_chunk; the epilogue reads it the same way).
                    const int sw = u & 7;
                    // The folded query decay * r~ goes out as fp16 times two powers of two: the one that brings the decay into
                    // [1, 2) and the row's own (the guess taken from |q| when the quad started: |r~| < 2^R_TARGET / q_scale).
                    // The guess is checked against the folded row: OR-ing the magnitudes' bits bounds the largest one from
                    // above, and if for any unit of the warp that bound reaches 2^(R_TARGET + 4) after scaling (keys longer
                    // than 1 or beta outside [0, 2] lengthened r~), the warp takes the row's true largest element instead.
                    // Either way the row stays far inside fp16's range.  The epilogue multiplies the accumulator by the
                    // reciprocals (and by that of the head's S_0 scale), exactly.
                    {
                        uint32_t orb = 0;
#pragma unroll
                        for (int e = 0; e < 4 * NCH; ++e) orb |= __float_as_uint(r[e].x) | __float_as_uint(r[e].y);
                        const bool suspect = !(__uint_as_float(orb & 0x7fffffffu) * q_scale < (float)(1 << (R_TARGET + 4)));
                        if (__any_sync(0xffffffffu, suspect)) {
                            uint32_t mx = 0;
#pragma unroll
                            for (int e = 0; e < 4 * NCH; ++e)
                                mx = max(mx, max(__float_as_uint(r[e].x) & 0x7fffffffu, __float_as_uint(r[e].y) & 0x7fffffffu));
#pragma unroll
                            for (int o = LPU / 2; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                            pow2_scale(__uint_as_float(mx), R_TARGET, q_scale, q_inv);
                        }
                    }
                    float d_scale, d_inv;
                    pow2_scale(decay, 0, d_scale, d_inv);
                    if (g == 0) inv_s[s * GN + u] = (q_inv * d_inv) * seg_inv_s0;
                    const float dcs = (decay * d_scale) * q_scale;
                    const float2 dc = make_float2(dcs, dcs);
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int ci = c * LPU + g;                 // elements [8 ci, 8 ci + 8)
                        float2 x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) x[e] = __fmul2_rn(r[4 * c + e], dc);
                        // fp16 operand rows: K blocks of 64 elements (128 bytes, 128-byte swizzle), one 16-byte chunk
                        // per lane and c; a warp's four rows are 512 consecutive bytes: no bank conflicts
                        uint8_t* row = R_s + (ci >> 3) * R_KB_STRIDE + u * 128;
                        *reinterpret_cast<uint4*>(row + (((ci & 7) ^ sw) << 4)) =
                            make_uint4(pack_f16x2(x[0].x, x[0].y), pack_f16x2(x[1].x, x[1].y), pack_f16x2(x[2].x, x[2].y),
                                       pack_f16x2(x[3].x, x[3].y));
                        float* crow = C_s + u * DV;
                        *reinterpret_cast<float4*>(crow + corr_chunk(2 * ci) * 4) =
                            make_float4(corr[4 * c].x, corr[4 * c].y, corr[4 * c + 1].x, corr[4 * c + 1].y);
                        *reinterpret_cast<float4*>(crow + corr_chunk(2 * ci + 1) * 4) =
                            make_float4(corr[4 * c + 2].x, corr[4 * c + 2].y, corr[4 * c + 3].x, corr[4 * c + 3].y);
                    }
                }
                if (DELTA && (grp & 1) == 0) {      // what the epilogue needs to form delta_t and o_t of this beam
                    uint8_t* ds = delta_s + s * DELTA_SLOT_BYTES;
                    const int bq = u >> 1;
#pragma unroll
                    for (int c = 0; c < NCH; ++c) *reinterpret_cast<uint4*>(ds + bq * (DV * 2) + (c * LPU + g) * 16) = cur.own.v[c];
                    if (g == 0) *reinterpret_cast<float4*>(ds + DELTA_BEAMS * (DV * 2) + bq * 16) = make_float4(cur.own.gate.x, cur.own.gate.y, kq, 0.f);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
                __syncwarp();
#ifdef ONELA_TEST_HOOKS
                if (g_hook_drop_full_arrival && blockIdx.x == 0 && warp == 0 && k == 0) continue;
#endif
                if (lane == 0) mbar_arrive(bar_full(s));
                TL(14, k);  // fold: rows written

                // The next quad's records of the levels that are NOT staged are gathered from global memory in the middle
                // of its dependent chain.  Where a level has little sharing (most of its records are used by one or two
                // beams: uniform parents) their lines are requested now, a whole quad ahead - the slot ids have arrived
                // by now; where many beams share few records the gathers hit L1/L2 anyway and the requests only cost
                // (measured: +6 % on 8 x 1024 beams with uniform parents, -3 % on the Zipf(1.5) stack if done always).
                // One request per lane: lane g of a unit asks for line g & 3 of the record of level
                // old - 1 - 2 p - (g >> 2), newest levels first.  (The segment's own staging layout is used for the
                // next quad: it differs only across a change of request, and a request is a hint.)
                if (AHEAD && n_ahead > 0 && k + 1 < n_quads) {
                    for (int p = 0; 2 * p < n_ahead; ++p) {
                        const int level = old - 1 - 2 * p - (g >> 2);
                        const int src = max(level, 0);
                        int32_t slot = 0;
#pragma unroll
                        for (int j = 0; j < NIDX; ++j) {
                            const int32_t x = __shfl_sync(0xffffffffu, idx_next.v[j], src & (LPU - 1), LPU);
                            if (j == src / LPU) slot = x;
                        }
                        if (level >= staged_levels && level < NIDX * LPU && ((info_sparse >> level) & 1)) {
                            const char* line = (g & 2) ? v_at(u1.h, slot) + (g & 1) * 128 : k_at(u1.h, slot) + (g & 1) * 128;
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
                        }
                    }
                }
            }
        };
        // little sharing somewhere in the first request's gathered levels: take the loop that requests lines ahead
        // (the requests of a batch follow one parent law as a rule; it is a hint either way)
        bool ahead = false;
        if (n_quads > 0) {
            const int sl0 = staged_levels_of(u0.req);
            ahead = old > sl0 && (info_sparse >> sl0) != 0;
        }
        if (ahead) fold_quads(std::true_type{});
        else fold_quads(std::false_type{});
    } else {
        // =============================== EPILOGUE (+ MMA issue, + preparation of the next segments) ===============================
        dependency_wait();
        const int quad = warp & 3;                    // tensor-memory lane quadrant of this warp
        const int i = quad * 32 + lane;               // output element (dv index) of this thread
        int staged_issued[2] = {0, 0};                // stagings requested per buffer (what teardown must wait for)
        // Stage the distinct records of segment `seg`: one 512-byte bulk copy per record, its gates by a plain load, one
        // record per lane.  Every lane arrives once, announcing the bytes it requested; its gate store is ordered
        // before the arrival.  The barrier completes even when nothing is staged.
        auto stage_segment = [&](int seg) {
            const int pair = pair_begin + seg, req = pair / a.H, h = pair - req * a.H;
            const int b = single ? 0 : (seg & 1);
            int levels, count;
            staging_of(req, levels, count);
            const long long plane_row0 = (long long)value_head(h) * a.arena_slots;
            const int li = (warp - FOLD_WARPS) * 32 + lane;
            if (li < count) {
                const long long slot = __ldg(a.ulist + req * a.ulist_req_stride + li), row = plane_row0 + slot;
                const uint32_t dst = smem_u32(stage + (b * STAGE_BUF + li) * REC_BYTES);
                if constexpr (GROUPED) {      // the two halves of the staged row come from the two planes
                    bulk_load(dst, k_at(h, slot), DK * 2, bar_stage(b));
                    bulk_load(dst + DK * 2, v_at(h, slot), DV * 2, bar_stage(b));
                } else {
                    bulk_load(dst, kv + row * REC_BYTES, REC_BYTES, bar_stage(b));
                }
                gates_s[b * STAGE_BUF + li] = __ldg(a.gates + row);
            }
            mbar_expect_tx(bar_stage(b), li < count ? REC_BYTES : 0);
            ++staged_issued[b];
        };
        // S_0 of segment `seg` (>= 1) into its tensor-memory buffer, by the four epilogue warps alone.
        auto prepare_s0 = [&](int seg) {
            load_s0(pair_begin + seg, seg & 1, 0, 1, seg + 1 < n_segs);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s0(seg & 1));
        };
        if (n_segs > 0) stage_segment(0);
        put_first_s0();
        if (n_segs > 1) {          // (doing this part later, or before the dependency wait with all warps, measured slower)
            stage_segment(1);
            prepare_s0(1);
        }

        // The first epilogue warp issues a group's 8 MMAs as soon as all its rows are written (never a fold warp:
        // whichever fold warp issued would be the last to finish its next quad).  It does so one group AHEAD: once
        // the tile of group k is complete (the named barrier below) it issues group k + 1 while the other three
        // warps store group k, so neither the issuing nor the MMAs' latency lies between two epilogues.
        auto issue_mma = [&](int gcount, int seg, bool seg_first) -> bool {     // warp FOLD_WARPS only; true: gave up
            const int s = gcount % SLOTS, use = gcount / SLOTS;
            int mma_failed = 0;
            if (lane == 0) {
                TL(20, gcount);  // issue: waiting for the rows
                bool ok = wait_or_abort(bar_full(s), use & 1, abort_flag);
                TL(21, gcount);  // issue: rows complete
                // segment 0's S_0 has a barrier of its own; segment seg >= 1 is use ((seg + 1) >> 1) - 1 of its
                // buffer's barrier
                if (ok && seg_first && seg >= 1) ok = wait_or_abort(bar_s0(seg & 1), (((seg + 1) >> 1) - 1) & 1, abort_flag);
                if (ok && gcount == 0) ok = wait_or_abort(bar_s0_first, 0, abort_flag);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (ok) {
                    constexpr uint32_t idesc = idesc_f16(GN);
                    const uint64_t bd = umma_desc(smem_u32(ring + s * SLOT_BYTES));
                    const uint32_t s0_at = tmem_base + S0_COL + (seg & 1) * 128;
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb)          // K block of 64 elements; 16 elements (32 bytes, 8 columns) per MMA
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_f16_ts(tmem_base + s * GN, s0_at + (kb * 4 + ks) * 8,
                                        bd + (uint64_t)((kb * R_KB_STRIDE + ks * 32) >> 4), idesc, (kb | ks) ? 1u : 0u);
                } else {
                    mma_failed = 1;
                }
                umma_commit(bar_done(s));   // arrives when the MMAs above have completed
                TL(22, gcount);  // issue: MMAs out
            }
            return __shfl_sync(0xffffffffu, mma_failed, 0) != 0;
        };
        // (request, head, group within the pair) of the group at hand, advanced without divisions
        int pair = pair_begin, req = pair / a.H, h = pair - req * a.H, gip = g_begin - pair * groups_per_pair;
        int issued = 0;                               // groups whose MMAs have been issued (first epilogue warp)
        // A warp that gives up (`fail`) never leaves on its own: it skips its work, raises the abort flag and keeps
        // arriving at the iteration's named barrier, whose OR makes all four warps leave in the same iteration.
        bool fail = false;
        auto give_up = [&]() {
            fail = true;
            if (lane == 0) *abort_flag = 1;
        };
        for (int gcount = 0; gcount < g_end - g_begin; ++gcount) {
            const int s = gcount % SLOTS, use = gcount / SLOTS;
            const int seg = pair - pair_begin;
            const bool seg_first = gcount == 0 || gip == 0;
            const bool has_next = gcount + 1 < g_end - g_begin;
            const bool next_first = gip + 1 == groups_per_pair;      // the next group opens a segment
            if (!fail && warp == FOLD_WARPS && issued == gcount) {
                if (issue_mma(gcount, seg, seg_first)) give_up();
                ++issued;
            }
            TL(30, gcount);  // epilogue: waiting for the accumulators
            if (!fail && !wait_or_abort(bar_done(s), use & 1, abort_flag)) give_up();
            TL(31, gcount);  // epilogue: accumulators complete
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float* C_s = reinterpret_cast<float*>(ring + s * SLOT_BYTES + R_BYTES);
            const int b0 = gip * BPG;
            const uint32_t taddr = tmem_base + s * GN + ((uint32_t)(quad * 32) << 16);
            float* A_s = reinterpret_cast<float*>(ring + s * SLOT_BYTES);   // the operand rows are dead once the MMAs have completed
            if (!fail) {
                // accumulator rows (dv) of this thread, all beams of the group, transposed into a tile laid out like
                // the corr tile, over the slot's operand rows (plain stores: nothing here waits for a shared-memory read)
                uint32_t v[GN];
#pragma unroll
                for (int c0 = 0; c0 < GN; c0 += 16) tmem_ld16(taddr + c0, v + c0);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int ip = corr_chunk(i >> 2) * 4 + (i & 3);   // where the corr tile keeps element i of a row
#pragma unroll
                for (int j = 0; j < GN; ++j) A_s[j * DV + ip] = __uint_as_float(v[j]);
            }
            // the four epilogue warps: tile complete - or somebody gave up, and then all four leave here together
            if (bar_or(1, 128, fail ? 1 : 0)) { dead = true; break; }
            TL(32, gcount);  // epilogue: tile transposed
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (warp == FOLD_WARPS) {
                // This warp's part of the slot is read out; the next group's MMAs go out now - unless that group
                // opens a segment whose S_0 this very iteration prepares below (a one-group segment).
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free(s));
                if (has_next && !(next_first && seg_first && seg >= 1)) {
                    if (issue_mma(gcount + 1, seg + (next_first ? 1 : 0), next_first)) give_up();   // carried to the next barrier
                    ++issued;
                }
            } else if constexpr (DELTA) {
                // Eq. 2 and 4 on the two projections of each beam (rows 2 j and 2 j + 1 of the tile):
                //   delta_t = beta_t (v_t - alpha_t S_{t-1} k_t) ,  o_t = alpha_t S_{t-1} q_t + delta_t (k_t . q_t) ;
                // the output row and the record's delta half (in the record dtype) leave as 16-byte stores
                const int et = (warp - FOLD_WARPS - 1) * 32 + lane;
                const uint8_t* ds = delta_s + s * DELTA_SLOT_BYTES;
                OutT* out0 = static_cast<OutT*>(a.out) + (((long long)req * a.W + b0) * a.H + h) * DV;
                char* rec0 = a.kv_out + ((long long)h * a.arena_slots + a.bases.base[req] + b0) * REC_BYTES + DK * 2;
#pragma unroll
                for (int it = 0; it < DELTA_BEAMS * 16 / 96; ++it) {
                    const int idx = it * 96 + et, j = idx >> 4, ch = idx & 15;
                    if (b0 + j < a.W) {
                        const int c0 = corr_chunk(2 * ch) * 4, c1 = corr_chunk(2 * ch + 1) * 4;
                        const float wq = inv_s[s * GN + 2 * j], wk = inv_s[s * GN + 2 * j + 1];
                        const float* Aq = A_s + (2 * j) * DV;
                        const float* Cq = C_s + (2 * j) * DV;
                        const float4 aq0 = *reinterpret_cast<const float4*>(Aq + c0), aq1 = *reinterpret_cast<const float4*>(Aq + c1);
                        const float4 cq0 = *reinterpret_cast<const float4*>(Cq + c0), cq1 = *reinterpret_cast<const float4*>(Cq + c1);
                        const float4 ak0 = *reinterpret_cast<const float4*>(Aq + DV + c0), ak1 = *reinterpret_cast<const float4*>(Aq + DV + c1);
                        const float4 ck0 = *reinterpret_cast<const float4*>(Cq + DV + c0), ck1 = *reinterpret_cast<const float4*>(Cq + DV + c1);
                        const float uq[8] = {fmaf(aq0.x, wq, cq0.x), fmaf(aq0.y, wq, cq0.y), fmaf(aq0.z, wq, cq0.z), fmaf(aq0.w, wq, cq0.w),
                                             fmaf(aq1.x, wq, cq1.x), fmaf(aq1.y, wq, cq1.y), fmaf(aq1.z, wq, cq1.z), fmaf(aq1.w, wq, cq1.w)};
                        const float uk[8] = {fmaf(ak0.x, wk, ck0.x), fmaf(ak0.y, wk, ck0.y), fmaf(ak0.z, wk, ck0.z), fmaf(ak0.w, wk, ck0.w),
                                             fmaf(ak1.x, wk, ck1.x), fmaf(ak1.y, wk, ck1.y), fmaf(ak1.z, wk, ck1.z), fmaf(ak1.w, wk, ck1.w)};
                        const float4 sc = *reinterpret_cast<const float4*>(ds + DELTA_BEAMS * (DV * 2) + j * 16);     // alpha_t, beta_t, k_t . q_t
                        float2 vx[4];
                        unpack8(*reinterpret_cast<const uint4*>(ds + j * (DV * 2) + ch * 16), vx);
                        const float vv[8] = {vx[0].x, vx[0].y, vx[1].x, vx[1].y, vx[2].x, vx[2].y, vx[3].x, vx[3].y};
                        float dl[8], o[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            dl[e] = sc.y * fmaf(-sc.x, uk[e], vv[e]);
                            o[e] = fmaf(dl[e], sc.z, sc.x * uq[e]);
                        }
                        store8<OutT>(out0 + (long long)j * a.H * DV + ch * 8, o);
                        store8<__nv_bfloat16>(reinterpret_cast<__nv_bfloat16*>(rec0 + (long long)j * REC_BYTES + ch * 16), dl);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free(s));
            } else {
                // coalesced stores by the other three warps: 16 lanes cover one beam's 128 outputs, 8 elements each
                const int et = (warp - FOLD_WARPS - 1) * 32 + lane;
                OutT* out0 = static_cast<OutT*>(a.out) + (((long long)req * a.W + b0) * a.H + h) * DV;
                float w8[GN * 16 / 96];                        // what undoes the scales of each row this thread stores
#pragma unroll
                for (int it = 0; it < GN * 16 / 96; ++it) w8[it] = inv_s[s * GN + ((it * 96 + et) >> 4)];
#pragma unroll
                for (int it = 0; it < GN * 16 / 96; ++it) {    // GN * 16 chunks of 16 bytes over 96 threads
                    const int idx = it * 96 + et, j = idx >> 4, ch = idx & 15;
                    if (b0 + j < a.W) {
                        const int o0 = j * DV + corr_chunk(2 * ch) * 4, o1 = j * DV + corr_chunk(2 * ch + 1) * 4;
                        const float4 x0 = *reinterpret_cast<const float4*>(C_s + o0), y0 = *reinterpret_cast<const float4*>(A_s + o0);
                        const float4 x1 = *reinterpret_cast<const float4*>(C_s + o1), y1 = *reinterpret_cast<const float4*>(A_s + o1);
                        const float w = w8[it];
                        const float o[8] = {fmaf(y0.x, w, x0.x), fmaf(y0.y, w, x0.y), fmaf(y0.z, w, x0.z), fmaf(y0.w, w, x0.w),
                                            fmaf(y1.x, w, x1.x), fmaf(y1.y, w, x1.y), fmaf(y1.z, w, x1.z), fmaf(y1.w, w, x1.w)};
                        store8<OutT>(out0 + (long long)j * a.H * DV + ch * 8, o);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free(s));
            }

            TL(33, gcount);  // epilogue: group stored / next group issued
            // Past the first group of segment seg >= 1 every MMA of segment seg - 1 has completed and the fold warps
            // have read its staging buffer out (they signal that): both are free for segment seg + 1.  (More groups
            // follow, so a warp that gives up here meets the others at the next iteration's barrier.)
            if (seg_first && seg >= 1 && seg + 1 < n_segs && !fail) {
                if (!wait_or_abort(bar_sfree((seg + 1) & 1), ((seg - 1) >> 1) & 1, abort_flag)) {
                    give_up();
                } else {
                    stage_segment(seg + 1);
                    prepare_s0(seg + 1);
                }
            }
            if (++gip == groups_per_pair) {
                gip = 0;
                ++pair;
                if (++h == a.H) { h = 0; ++req; }
            }
        }
        if (fail) dead = true;
        if (dead && lane == 0) *abort_flag = 1;
        // A CTA must not exit with bulk copies still landing in its shared memory: after an abort nobody may have
        // waited for the stagings requested last.
        if (*abort_flag && warp == FOLD_WARPS && lane == 0) {
            for (int b = 0; b < 2; ++b)
                if (staged_issued[b] > 0) mbar_wait(bar_stage(b), (staged_issued[b] - 1) & 1);
        }
    }
    if (dead && lane == 0) {
        *abort_flag = 1;
        if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)blockIdx.x;
    }

#ifdef ONELA_WS_TL
    TL(40, 0);  // role done
    if (lane == 0 && tl_role >= 0) {
        for (int i = 0; i < tl_n; ++i) g_ws_tl[tl_role * TL_CAP + i] = tl_s[tl_role * TL_CAP + i];
        g_ws_tl_n[tl_role] = tl_n;
    }
#endif
    // nor with the fold warps' own async copies in flight
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

int sm_count_ws() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// Contiguous group ranges for the CTAs.  A CTA's cost is counted as group_cost * groups + seg_cost * segments (starting
// a segment: S_0 reloaded, staging refilled, the ring's overlap lost for a moment) and the smallest bound T is searched
// for which a greedy fill needs no more CTAs than there are SMs.  Returns the number of CTAs used.
// The costs, in units of ~500 cycles, follow what the kernel measures on the beam-512 stack: a group takes ~4000
// cycles plus ~500 per chain level beyond the first; starting a segment ~6000 at depth <= 3 (where whole (request,
// head) pairs per CTA, 128 x 11 groups, beat 141 x 10 groups over two segments by 0.6-1.5 us) and ~3000 deeper (where
// the shorter CTA wins by 0.6-2.5 us).
struct PartitionCost {
    int group, seg;
};
#ifndef ONELA_SEG_SHALLOW
#define ONELA_SEG_SHALLOW 12
#endif
#ifndef ONELA_SEG_DEEP
#define ONELA_SEG_DEEP 6
#endif
#ifndef ONELA_SHALLOW_DEPTH
#define ONELA_SHALLOW_DEPTH 3
#endif
PartitionCost partition_cost(int depth) {
    return {8 + (depth > 1 ? depth - 1 : 0), depth <= ONELA_SHALLOW_DEPTH ? ONELA_SEG_SHALLOW : ONELA_SEG_DEEP};
}
int greedy_fill(int total_groups, int gpp, int limit, int max_ctas, PartitionCost c, int32_t* begin) {
    int n = 0, gi = 0;
    while (gi < total_groups) {
        if (n == max_ctas) return max_ctas + 1;
        if (begin) begin[n] = gi;
        int cost = 0;
        bool any = false;
        while (gi < total_groups) {
            const int pair_end = (gi / gpp + 1) * gpp;
            const int room = (limit - cost - c.seg) / c.group;     // groups of this segment that still fit
            if (room <= 0) break;
            const int take = room < pair_end - gi ? room : pair_end - gi;
            gi += take;
            cost += c.seg + take * c.group;
            any = true;
            if (gi < pair_end) break;
        }
        if (!any) return max_ctas + 1;   // the bound does not admit a single group
        ++n;
    }
    if (begin) begin[n] = total_groups;
    return n;
}
int make_partition(int total_groups, int gpp, int sms, PartitionCost c, Partition* part) {
    int lo = c.seg + c.group, hi = c.seg * (total_groups / gpp + 2) + c.group * total_groups;
    while (lo < hi) {
        const int mid = (lo + hi) / 2;
        if (greedy_fill(total_groups, gpp, mid, sms, c, nullptr) <= sms) hi = mid;
        else lo = mid + 1;
    }
    return greedy_fill(total_groups, gpp, lo, sms, c, part->begin);
}

template <typename OutT, bool GROUPED, bool FUSED, bool DELTA = false>
cudaError_t launch_ws_t(const DecodeArgs& a, cudaStream_t stream) {
    auto kern = decode_ws_kernel<OutT, GROUPED, FUSED, DELTA>;
    constexpr int SMEM_BYTES = DELTA ? SMEM_BYTES_DELTA : onela::SMEM_BYTES;
    constexpr int GN = DELTA ? DELTA_BEAMS : onela::GN;      // beams per group (a delta-record group has two rows per beam)
    // One-time set-up per device (function attributes belong to a device's context); host threads may share it.
    constexpr int MAX_DEVICES = 64;
    static std::mutex setup_mutex;
    static int sms_of[MAX_DEVICES] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    int sms;
    {
        std::lock_guard<std::mutex> lock(setup_mutex);
        if (sms_of[dev] == 0) {
            const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            if (e != cudaSuccess) return e;
            const int n = sm_count_ws();
            sms_of[dev] = n > MAX_CTAS ? MAX_CTAS : n;
        }
        sms = sms_of[dev];
    }
    const int groups_per_pair = (a.W + GN - 1) / GN;
    const int total_groups = a.req_count * a.H * groups_per_pair;
    static thread_local Partition part;          // the last launch's partition, reused while the shape stays
    static thread_local int part_total = -1, part_gpp = -1, part_sms = -1, part_group = -1, part_seg = -1, part_ctas = 0;
    const PartitionCost cost = partition_cost(a.depth);
    if (part_total != total_groups || part_gpp != groups_per_pair || part_sms != sms || part_group != cost.group ||
        part_seg != cost.seg) {
        part_ctas = make_partition(total_groups, groups_per_pair, sms, cost, &part);
        part_total = total_groups; part_gpp = groups_per_pair; part_sms = sms;
        part_group = cost.group; part_seg = cost.seg;
    }
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
    return cudaLaunchKernelEx(&cfg, kern, a, part, groups_per_pair);
}

}  // namespace

#ifdef ONELA_WS_TL
extern "C" int onela_debug_ws_timeline_cta(int cta) { return (int)cudaMemcpyToSymbol(g_ws_tl_cta, &cta, sizeof(int)); }
extern "C" int onela_debug_ws_timeline(unsigned long long* out_host, int* counts_host) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(counts_host, g_ws_tl_n, 3 * sizeof(int));
    cudaMemcpyFromSymbol(out_host, g_ws_tl, sizeof(unsigned long long) * 3 * TL_CAP);
    const int zero[3] = {0, 0, 0};
    cudaMemcpyToSymbol(g_ws_tl_n, zero, sizeof(zero));
    return TL_CAP;
}
#endif

#ifdef ONELA_TEST_HOOKS
extern "C" int onela_testhook_drop_full_arrival(int on) {
    return (int)cudaMemcpyToSymbol(g_hook_drop_full_arrival, &on, sizeof(int));
}
#endif

int make_decode_partition(int total_groups, int groups_per_pair, int sms, int group_cost, int seg_cost, DecodePartition* part) {
    return make_partition(total_groups, groups_per_pair, sms > MAX_CTAS ? MAX_CTAS : sms, PartitionCost{group_cost, seg_cost}, part);
}
int decode_sm_count() { return sm_count_ws(); }

bool decode_sm100_supported(int32_t dk, int32_t dv, int32_t rec_dtype) {
    // value widths of 256 and 512 run as two or four value heads of 128 outputs that share the key head's fold
    return dk == 128 && (dv == 128 || dv == 256 || dv == 512) && rec_dtype == ONELA_DTYPE_BF16;
}

cudaError_t launch_decode_sm100_ws(const DecodeArgs& a, int32_t out_dtype, bool grouped, bool delta_records, cudaStream_t stream) {
    // one instantiation per (output type, grouped value heads, append fused in): a launch runs only the code it needs
    const bool fused = a.k_in != nullptr;
    const bool bf16 = out_dtype == ONELA_DTYPE_BF16;
    if (delta_records) {
        if (grouped || !fused) return cudaErrorInvalidValue;
        return bf16 ? launch_ws_t<__nv_bfloat16, false, true, true>(a, stream) : launch_ws_t<float, false, true, true>(a, stream);
    }
    if (grouped) {
        if (fused) return bf16 ? launch_ws_t<__nv_bfloat16, true, true>(a, stream) : launch_ws_t<float, true, true>(a, stream);
        return bf16 ? launch_ws_t<__nv_bfloat16, true, false>(a, stream) : launch_ws_t<float, true, false>(a, stream);
    }
    if (fused) return bf16 ? launch_ws_t<__nv_bfloat16, false, true>(a, stream) : launch_ws_t<float, false, true>(a, stream);
    return bf16 ? launch_ws_t<__nv_bfloat16, false, false>(a, stream) : launch_ws_t<float, false, false>(a, stream);
}

}  // namespace onela
