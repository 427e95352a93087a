// Fused decode kernel for B200 (sm_100a) for beams whose chains share most of their older records
// (dk = dv = 128, bf16 records): every chain level but the newest is applied on the tensor cores.
//
// The method (Section 3.2, Eq. 1-4 read backward): with A_j = alpha_j (I - beta_j k_j k_j^T) the output of a beam is
//   o = S_0 (A_0 ... A_t q) + sum_j beta_j c_j v_j ,  c_j = k_j . r_j ,  r_t = q ,  r_{j-1} = A_j r_j .
// Only the newest record (the beam's own) is folded per beam on the CUDA cores: rho = alpha_t (q - beta_t c_t k_t).
// The older records of a (request, head) form a small tree of DISTINCT nodes (the ancestry index lists them); for
// a chain kappa_0 (oldest) .. kappa_{m-1} (the parent) the recursion unrolls, without the decays, to
//   chat_l = k_l . rho - sum_{l' > l} beta_l' chat_l' (k_l . k_l') ,                       (a triangular solve)
//   o = D S_0 rho + sum_l w_l (v_l - e_l S_0 k_l) + beta_t c_t v_t ,
//   w_l = beta_l d_l chat_l ,  d_l = prod_{l' > l} alpha_l' ,  D = prod_l alpha_l ,  e_l = prod_{l' <= l} alpha_l'
// where e_l and u_l = v_l - e_l S_0 k_l belong to the NODE (a node's ancestors are unique), not to the beam.  So
//   per segment (request, head):  P = S_0 K^T and the Gram block K K_deep^T on the tensor cores (K: the nodes' keys),
//                                 U = [u_kappa] into tensor memory, the chain dot products k_l . k_l' into a table;
//   per group of 48 beams:        [S_0 ; K] . R^T (R: the 48 folded queries), the 48 small triangular solves on
//                                 CUDA cores (one thread per beam, a few dozen FMAs), U . W^T (W: the weights w_l,
//                                 one row per beam, zero outside its chain), and the epilogue
//                                 o = coefA acc1 + coefB acc2 + beta_t c_t v_t.
// The per-level cost on the CUDA cores falls from a 128-element dot and two 128-element updates per beam to one
// multiply-add per beam and level pair.
//
// One persistent CTA per SM, 20 warps, three roles coupled by mbarriers over a ring of two 48-beam slots:
//   * 12 FOLD warps (8 lanes per unit, 4 units per warp and group): newest record, operand row (fp16, scaled by a
//     power of two taken from the row itself), the raw value row for the epilogue, the fused append.
//   * 4 EPILOGUE warps: issue [S_0 ; K] . R^T one group ahead, combine the two accumulators, transpose through
//     shared memory, add the newest record's term, store.
//   * 4 SOLVER warps: pick each beam's chain entries out of K . R^T (lane = node), solve, write W, issue U . W^T.
// Both back-side teams build a segment's tables before its first group.  Every wait on an mbarrier is bounded and
// gives up when the CTA's abort flag is raised; a warp that gives up keeps arriving at its team's named barriers
// (whose OR makes the team leave together), records ONELA_E_TIMEOUT, and the CTA frees its tensor memory.
#include <mutex>

#include "onela_internal.h"
#include "onela_layout.cuh"
#include "onela_sm100.cuh"

namespace onela {

namespace {

using namespace sm100;

constexpr int FOLD_WARPS = 12;
constexpr int LPU = 8;                              // lanes per (beam, head) unit
constexpr int UPW = 32 / LPU;                       // units per fold warp and group
constexpr int NCH = 16 / LPU;                       // 16-byte chunks per lane per 256-byte vector
constexpr int EPI_WARP0 = FOLD_WARPS;               // warps 12..15: epilogue team
constexpr int SOL_WARP0 = FOLD_WARPS + 4;           // warps 16..19: solver team
constexpr int ISS_WARP = SOL_WARP0 + 3;             // the last solver warp (idle during the solves) issues [S_0 ; K] . R^T
constexpr int THREADS = (FOLD_WARPS + 8) * 32;      // 640
constexpr int GN = FOLD_WARPS * UPW;                // beams per group = MMA N (48)
constexpr int MAXN = WY_MAX_NODES, MAXD = WY_MAX_DEEP, MAXL = WY_MAX_LEVELS;
constexpr int SLOTS = 2;                            // operand rows, weight tiles, U . W^T accumulators
constexpr int VSLOTS = 3;                           // value rows, per-beam scalars, S_0 . R^T accumulators (live until the epilogue)
constexpr int MAXW = 1024;                          // beams per request whose chain nodes fit the per-segment table

// ---- shared memory ----
constexpr int R_KB_STRIDE = GN * 128;               // bytes between the two K blocks (64 fp16) of the operand rows
constexpr int R_BYTES = 2 * R_KB_STRIDE;            // folded queries, K-major, 128-byte swizzle
constexpr int W_KBLOCKS = (MAXN + 63) / 64;
constexpr int W_KB_STRIDE = GN * 128;
constexpr int W_BYTES = W_KBLOCKS * W_KB_STRIDE;    // weights, K-major over the nodes, 128-byte swizzle
constexpr int T_BYTES = GN * DV * 4;                // transposed outputs, over the operand rows and the weights (dead by then)
constexpr int VT_BYTES = GN * DV * 2;               // the group's own value rows, raw bf16
// [operand rows x 2][transposed tile][weights x 2][value rows x 3][node keys][fold warps' stages][tables]
constexpr int OFF_R = 0;
constexpr int OFF_T = OFF_R + SLOTS * R_BYTES;
constexpr int OFF_W = OFF_T + T_BYTES;
constexpr int OFF_V = OFF_W + SLOTS * W_BYTES;
constexpr int OFF_A = OFF_V + VSLOTS * VT_BYTES;
constexpr int A_KB_STRIDE = MAXN * 128;             // node keys as fp16, K-major, 128-byte swizzle, row = node
constexpr int A_BYTES = 2 * A_KB_STRIDE;
constexpr int VS_BYTES = MAXN * DV * 2;             // set-up only: node values, raw bf16, row = node, over the transposed tile
                                                    // and the first weight tile
constexpr int OFF_HEADS = OFF_A + A_BYTES;
constexpr int HEAD_BYTES = UPW * (REC_BYTES + DK * 2);
constexpr int HEADS_TOTAL = FOLD_WARPS * HEAD_BYTES;
static_assert(VS_BYTES <= T_BYTES + W_BYTES, "the node values lie over the transposed tile and the first weight tile");
static_assert(OFF_T % 1024 == 0 && OFF_W % 1024 == 0 && OFF_A % 1024 == 0 && W_BYTES % 1024 == 0 && R_BYTES % 1024 == 0 &&
              A_KB_STRIDE % 1024 == 0 && R_KB_STRIDE % 1024 == 0, "swizzle atoms");
constexpr int HI_ROW0 = 64;                         // nodes 128.. are rows 64.. of the second key tile: tensor-memory lanes 64..95
static_assert(HI_ROW0 * 128 + A_KB_STRIDE + 128 * 128 <= A_BYTES + HEADS_TOTAL, "second key tile's over-read stays inside shared memory");
static_assert(128 * 128 <= W_BYTES, "the Gram bounce buffer fits the second weight tile");

struct Misc {
    float2 gates[MAXN];            // (alpha, beta) of the nodes
    float ne[MAXN];                // e_kappa / (S_0 scale)
    alignas(16) float ld[MAXN][MAXL];          // ld[kappa][l] = k_kappa . k_(ancestor of kappa at level l), l < level(kappa)
    alignas(8) uint8_t anc[MAXN][MAXL];       // ancestor of kappa at level l
    uint8_t lvl[MAXN];
    alignas(16) uint8_t sg[MAXL][MAXW + 64];   // node of beam b's chain at level l (whole request; idle beams shadow the last)
    alignas(16) float gout[SLOTS][MAXL][GN];   // k_node . (operand row of beam u) for the chain nodes of the group's beams
    alignas(16) float fA[VSLOTS][GN];          // fold warps: alpha_t / (row scale)
    float wt[VSLOTS][GN];                      // fold warps: beta_t c_t
    alignas(16) float cA[VSLOTS][GN];          // solver: coefficient of the S_0 accumulator
    alignas(16) float cB[VSLOTS][GN];          // solver: coefficient of the U accumulator
    uint32_t umax[24];
    alignas(8) uint64_t bars[24];
    uint32_t tmem_slot;
    int abort_flag;
};
constexpr int MISC_BYTES = (sizeof(Misc) + 127) & ~127;
#ifdef ONELA_WY_TL
constexpr int TL_BYTES = 4 * 200 * 8;
#else
constexpr int TL_BYTES = 0;
#endif
constexpr int SMEM_BYTES = OFF_HEADS + HEADS_TOTAL + MISC_BYTES + TL_BYTES + 1024;
static_assert(SMEM_BYTES <= 232448, "shared memory per CTA");

// ---- tensor memory columns ----
constexpr uint32_t ACC1_COL = 0;                    // + (g % 3) * GN : S_0 . R^T
constexpr uint32_t GLO_COL = 144;                   // K[0..127] . R^T (read out by the solver team before the next group's goes in)
constexpr uint32_t GHI_COL = 192;                   // K[128..] . R^T
constexpr uint32_t ACC2_COL = 240;                  // + (g % 2) * GN : U . W^T
constexpr uint32_t S0_COL = 336;                    // 64 columns: S_0 as fp16 pairs
constexpr uint32_t U_COL = 400;                     // MAXN / 2 columns: U as fp16 pairs
constexpr uint32_t PACC_COL = 0;                    // set-up only: S_0 K^T (up to MAXN columns)
constexpr uint32_t GRAM_LO_COL = 160;               // set-up only: K[0..127] K_deep^T (up to MAXD columns)
constexpr uint32_t GRAM_HI_COL = 224;               // set-up only: K[128..] K_deep^T
constexpr uint32_t TMEM_COLS = 512;
static_assert(VSLOTS * GN <= GLO_COL && ACC2_COL + SLOTS * GN <= S0_COL && U_COL + MAXN / 2 <= 512, "tensor-memory map");
static_assert(PACC_COL + MAXN <= GRAM_LO_COL && GRAM_LO_COL + MAXD <= GRAM_HI_COL && GRAM_HI_COL + MAXD <= S0_COL, "set-up accumulators");
static_assert(MAXL == 8, "the solve is written out for eight levels");
constexpr int R_TARGET = 8;                         // a scaled operand row's largest element lies in [2^8, 2^9)
constexpr int W_TARGET = 7;
constexpr int U_TARGET = 12;                        // the bound on |u| times the scale lies in [2^12, 2^13)

#ifdef ONELA_WY_TL
// Debug builds only: clock stamps of CTA 0's role milestones, kept in shared memory and written out when the CTA
// ends (never compiled into the product library).
constexpr int TL_CAP = 200;
__device__ unsigned long long g_wy_tl[4 * TL_CAP];
__device__ int g_wy_tl_n[4];
#define TL(ev, g)                                                                                         \
    do {                                                                                                  \
        if (lane == 0 && tl_role >= 0 && tl_n < TL_CAP)                                                   \
            tl_s[tl_role * TL_CAP + tl_n++] = ((unsigned long long)(ev) << 56) | ((unsigned long long)((g) & 0xff) << 48) | \
                                              ((unsigned long long)clock64() & 0xffffffffffffull);         \
    } while (0)
#else
#define TL(ev, g) do { } while (0)
#endif

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (int i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63 && *abort_flag) return false;
#ifdef ONELA_WY_NAP
        __nanosleep(ONELA_WY_NAP);
#endif
    }
    return false;
}
// The same for a whole warp: every lane gets the same answer, so warp-collective instructions that follow stay aligned.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, wait_or_abort(bar, parity, abort_flag) ? 1 : 0) != 0;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void named_bar(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ int corr_chunk(int q) { return q ^ ((q >> 3) & 1); }
// two packed bf16 -> two packed fp16 (exact for magnitudes inside fp16's normal range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    return pack_f16x2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

template <typename OutT, bool FUSED>
__global__ void __launch_bounds__(THREADS, 1) decode_wy_kernel(const __grid_constant__ DecodeArgs a,
                                                               const __grid_constant__ DecodePartition part,
                                                               int groups_per_pair) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* A_s = smem + OFF_A;
    uint8_t* VS_s = smem + OFF_T;                     // set-up only
    uint8_t* T_raw = smem + OFF_T;
    uint8_t* heads = smem + OFF_HEADS;
    Misc& mi = *reinterpret_cast<Misc*>(heads + HEADS_TOTAL);
    volatile int* abort_flag = &mi.abort_flag;
#ifdef ONELA_WY_TL
    unsigned long long* tl_s = reinterpret_cast<unsigned long long*>(heads + HEADS_TOTAL + MISC_BYTES);
    const int tl_role = blockIdx.x != 0 ? -1 : warp == 0 ? 0 : warp == EPI_WARP0 ? 1 : warp == SOL_WARP0 ? 2 : warp == ISS_WARP ? 3 : -1;
    int tl_n = 0;
#endif
    // Group g of the CTA uses operand rows / weight tile / U . W^T accumulator g % 2 and value rows / scalars /
    // S_0 . R^T accumulator g % 3.
    auto bar_full = [&](int s) { return smem_u32(mi.bars + s); };          // [2] fold warps -> issuer (12 arrivals)
    auto bar_done1 = [&](int s) { return smem_u32(mi.bars + 2 + s); };     // [2] [S_0 ; K] . R^T complete (commit)
    auto bar_done2 = [&](int s) { return smem_u32(mi.bars + 4 + s); };     // [2] U . W^T complete (commit)
    auto bar_free = [&](int v) { return smem_u32(mi.bars + 6 + v); };      // [3] epilogue done with group (4 arrivals)
    const uint32_t bar_s0_first = smem_u32(mi.bars + 10);
    const uint32_t bar_setup_mma = smem_u32(mi.bars + 11);
    const uint32_t bar_team = smem_u32(mi.bars + 12);                      // the eight back-side warps
    auto slot_R = [&](int s) { return smem + OFF_R + s * R_BYTES; };
    auto slot_W = [&](int s) { return smem + OFF_W + s * W_BYTES; };
    auto slot_V = [&](int v) { return smem + OFF_V + v * VT_BYTES; };

    if (tid == 0) {
        for (int s = 0; s < SLOTS; ++s) {
            mbar_init(bar_full(s), FOLD_WARPS);
            mbar_init(bar_done1(s), 1);
            mbar_init(bar_done2(s), 1);
        }
        for (int v = 0; v < VSLOTS; ++v) mbar_init(bar_free(v), 4);
        mbar_init(bar_s0_first, 16);
        mbar_init(bar_setup_mma, 1);
        mbar_init(bar_team, 8);
        mi.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&mi.tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = mi.tmem_slot;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int g_begin = part.begin[blockIdx.x], g_end = part.begin[blockIdx.x + 1];
    const int pair_begin = g_begin / groups_per_pair;
    const int n_segs = g_begin < g_end ? (g_end - 1) / groups_per_pair - pair_begin + 1 : 0;
    const int m = a.depth - 1;                         // chain levels older than a beam's own record
    const char* kv = a.kv;
    const __nv_bfloat16* qbase = static_cast<const __nv_bfloat16*>(a.q);
    const int grp = lane / LPU, g = lane % LPU;
    bool dead = false;

    // The first segment's S_0: requested by the first sixteen warps before the launch's dependencies are waited for
    // (the store is written only by the state calls, and a reorder launch always separates those from a decode),
    // put into tensor memory as fp16 times the head's power-of-two scale.
    const bool s0_mine = warp < 16;
    float4 s0_first[8];
    float s0_first_scale = 1.f;
    if (n_segs > 0 && s0_mine) {
        const int req = pair_begin / a.H, h = pair_begin - req * a.H;
        s0_first_scale = __ldg(a.s0_scale + req * a.s0_scale_req_stride + h);
        const float* row = a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK) + (long long)((warp & 3) * 32 + lane) * DK + (warp >> 2) * 32;
#pragma unroll
        for (int c = 0; c < 8; ++c) s0_first[c] = __ldg(reinterpret_cast<const float4*>(row) + c);
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
    auto dependency_wait = [&]() { asm volatile("griddepcontrol.wait;" ::: "memory"); };

    if (warp < FOLD_WARPS) {
        // =============================== FOLD (newest record only) ===============================
        const int n_quads = g_end - g_begin;
        uint8_t* my_heads = heads + warp * HEAD_BYTES;
        struct Unit { int req, h, gip; };
        auto beam_of = [&](const Unit& u) { return u.gip * GN + UPW * warp + grp; };
        auto live_beam = [&](const Unit& u) { return min(beam_of(u), a.W - 1); };   // idle units shadow a live beam
        auto next_unit = [&](Unit u) {
            if (++u.gip == groups_per_pair) {
                u.gip = 0;
                if (++u.h == a.H) { u.h = 0; ++u.req; }
            }
            return u;
        };
        Unit u0;
        {
            const int pair = g_begin / groups_per_pair;
            u0.req = pair / a.H;
            u0.h = pair - u0.req * a.H;
            u0.gip = g_begin - pair * groups_per_pair;
        }
        auto in_row = [&](const Unit& u, int bb) { return ((long long)u.req * a.W + bb) * a.H + u.h; };
        auto arena_row = [&](const Unit& u, int bb) { return (long long)u.h * a.arena_slots + a.bases.base[u.req] + bb; };
        auto request_heads = [&](const Unit& n) {        // the 128-byte lines of a quad's heads, into L2
            if (lane < UPW * 6) {
                const int un = lane / 6, item = lane % 6;
                const int b2 = min(n.gip * GN + UPW * warp + un, a.W - 1);
                const long long row2 = in_row(n, b2);
                const char* p2 = item < 2 ? reinterpret_cast<const char*>(qbase) + row2 * (DK * 2)
                                 : FUSED  ? (item < 4 ? static_cast<const char*>(a.k_in) + row2 * (DK * 2)
                                                      : static_cast<const char*>(a.v_in) + row2 * (DV * 2))
                                          : kv + arena_row(n, b2) * REC_BYTES + (item < 4 ? 0 : DK * 2);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p2 + (item & 1) * 128));
            }
        };
        auto issue_head = [&](const Unit& u) {
            const uint32_t dst = smem_u32(my_heads);
            const int bb = live_beam(u);
            const long long row = in_row(u, bb);
            const char* qr = reinterpret_cast<const char*>(qbase + row * DK) + g * 16;
            const char *kr, *vr;
            if (FUSED) {
                kr = static_cast<const char*>(a.k_in) + row * (DK * 2) + g * 16;
                vr = static_cast<const char*>(a.v_in) + row * (DV * 2) + g * 16;
            } else {
                kr = kv + arena_row(u, bb) * REC_BYTES + g * 16;
                vr = kr + DK * 2;
            }
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                cp_async16(dst + grp * REC_BYTES + (c * LPU + g) * 16, kr + c * LPU * 16);
                cp_async16(dst + grp * REC_BYTES + (16 + c * LPU + g) * 16, vr + c * LPU * 16);
                cp_async16(dst + UPW * REC_BYTES + grp * (DK * 2) + (c * LPU + g) * 16, qr + c * LPU * 16);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        auto load_gate = [&](const Unit& u) {
            const int bb = live_beam(u);
            if (!FUSED) return __ldg(a.gates + arena_row(u, bb));
            const long long row = in_row(u, bb);
            return make_float2(__ldg(a.alpha_in + row), __ldg(a.beta_in + row));
        };
        float2 gate0 = make_float2(1.f, 0.f), gate1 = gate0;
        Unit u1 = next_unit(u0), u2 = next_unit(u1);
        if (n_quads > 0) request_heads(u0);
        dependency_wait();
        if (n_quads > 0) {
            issue_head(u0);
            gate0 = load_gate(u0);
            if (1 < n_quads) gate1 = load_gate(u1);
        }
        put_first_s0();
        for (int k = 0; k < n_quads && !dead; ++k, u0 = u1, u1 = u2, u2 = next_unit(u2)) {
            const int s = k % SLOTS, vs = k % VSLOTS;
            TL(1, k);   // fold: quad start
            const int u = UPW * warp + grp;                  // row of this unit in the group
            const int bb = live_beam(u0);
            uint4 kq[NCH], vq[NCH], qq[NCH];
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            {
                const uint4* rec = reinterpret_cast<const uint4*>(my_heads + grp * REC_BYTES) + g;
                const uint4* qv = reinterpret_cast<const uint4*>(my_heads + UPW * REC_BYTES + grp * (DK * 2)) + g;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    kq[c] = rec[c * LPU];
                    vq[c] = rec[16 + c * LPU];
                    qq[c] = qv[c * LPU];
                }
            }
            const float2 gate = gate0;
            if (k + 1 < n_quads) issue_head(u1);
            if (FUSED && beam_of(u0) < a.W) {   // the append: this beam's record goes to its arena slot, bit for bit
                const long long arow = arena_row(u0, bb);
                uint4* dst = reinterpret_cast<uint4*>(a.kv_out + arow * REC_BYTES) + g;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    dst[c * LPU] = kq[c];
                    dst[16 + c * LPU] = vq[c];
                }
                if (g == 0) a.gates_out[arow] = gate;
            }
            gate0 = gate1;
            if (k + 2 < n_quads) gate1 = load_gate(u2);

            // c_t = k_t . q ;  x = q - beta_t c_t k_t  (alpha_t rides in the scalar handed to the solver)
            float2 r[4 * NCH], kx[4 * NCH];
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                unpack8(qq[c], r + 4 * c);
                unpack8(kq[c], kx + 4 * c);
            }
            float2 d0 = make_float2(0.f, 0.f), d1 = make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 4 * NCH; e += 2) {
                d0 = __ffma2_rn(kx[e], r[e], d0);
                d1 = __ffma2_rn(kx[e + 1], r[e + 1], d1);
            }
            float dot = (d0.x + d0.y) + (d1.x + d1.y);
#pragma unroll
            for (int o = LPU / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            const float bc = gate.y * dot;
            const float2 nbc2 = make_float2(-bc, -bc);
            uint32_t mx = 0;                                 // largest magnitude of the row, as bits
#pragma unroll
            for (int e = 0; e < 4 * NCH; ++e) {
                r[e] = __ffma2_rn(kx[e], nbc2, r[e]);
                mx = max(mx, max(__float_as_uint(r[e].x) & 0x7fffffffu, __float_as_uint(r[e].y) & 0x7fffffffu));
            }
#pragma unroll
            for (int o = LPU / 2; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float r_scale, r_inv;
            pow2_scale(__uint_as_float(mx), R_TARGET, r_scale, r_inv);

            TL(2, k);   // fold: arithmetic done, waiting for the buffers
            // the operand rows are free once the MMAs of group k - 2 have read them; the value rows and scalars once the
            // epilogue of group k - 3 has
            if (k >= SLOTS && !wait_or_abort(bar_done1(s), ((k / SLOTS) - 1) & 1, abort_flag)) { dead = true; break; }
            if (k >= VSLOTS && !wait_or_abort(bar_free(vs), ((k / VSLOTS) - 1) & 1, abort_flag)) { dead = true; break; }
            TL(3, k);   // fold: buffers free
            uint8_t* R_s = slot_R(s);
            uint8_t* V_s = slot_V(vs);
            const int sw = u & 7;
            const float2 sc2 = make_float2(r_scale, r_scale);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int ci = c * LPU + g;                 // elements [8 ci, 8 ci + 8)
                float2 x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = __fmul2_rn(r[4 * c + e], sc2);
                uint8_t* row = R_s + (ci >> 3) * R_KB_STRIDE + u * 128;
                *reinterpret_cast<uint4*>(row + (((ci & 7) ^ sw) << 4)) =
                    make_uint4(pack_f16x2(x[0].x, x[0].y), pack_f16x2(x[1].x, x[1].y), pack_f16x2(x[2].x, x[2].y),
                               pack_f16x2(x[3].x, x[3].y));
                *reinterpret_cast<uint4*>(V_s + u * (DV * 2) + ci * 16) = vq[c];
            }
            if (g == 0) {
                mi.fA[vs][u] = gate.x * r_inv;
                mi.wt[vs][u] = bc;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full(s));
            TL(4, k);   // fold: full arrived
        }
    } else {
        // =============================== BACK SIDE: epilogue team and solver team ===============================
        // What the set-up reads (index arrays, S_0, records of earlier decode calls) was written at least two launches
        // ago when the host says so; the epilogue team still waits for the predecessor before its first store.
        if (!a.early_ok) dependency_wait();
        const bool epi = warp < SOL_WARP0;
        const int quad = warp & 3;                    // tensor-memory lane quadrant of this warp
        const int row_i = quad * 32 + lane;           // tensor-memory lane of this thread
        const uint32_t lane_bits = (uint32_t)(quad * 32) << 16;
        const int tb = tid - EPI_WARP0 * 32;          // 0 .. 255
        const int bw = warp - EPI_WARP0;              // 0 .. 7
        bool fail = false;
        auto give_up = [&]() {
            fail = true;
            if (lane == 0) *abort_flag = 1;
        };
        uint32_t team_phase = 0;
        // Barrier over the eight back-side warps, bounded; false when somebody has given up.
        auto team_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_team);
            const bool ok = warp_wait(bar_team, team_phase & 1, abort_flag);
            ++team_phase;
            return __all_sync(0xffffffffu, (ok && !*abort_flag) ? 1 : 0) != 0;
        };
        constexpr uint32_t idesc_g = idesc_f16(GN);
        int gcount = 0;                                // groups of this CTA handled so far (both teams count alike)

        for (int seg = 0; seg < n_segs && !fail && !dead; ++seg) {
            const int pair = pair_begin + seg, req = pair / a.H, h = pair - req * a.H;
            const int seg_g0 = max(g_begin, pair * groups_per_pair), seg_g1 = min(g_end, (pair + 1) * groups_per_pair);
            const int32_t* uoff = a.uoff + req * a.uoff_req_stride;
            const int32_t* ulist = a.ulist + req * a.ulist_req_stride;
            const int32_t* urep = a.urep + req * a.ulist_req_stride;
            const int32_t* sidx = a.sidx + req * a.sidx_req_stride;
            const long long plane_row0 = (long long)h * a.arena_slots;
            const int n = __ldg(uoff + m), nd = __ldg(uoff + m - 1);        // nodes, and nodes older than the parents
            const int n16 = (n + 15) & ~15, nd16 = (nd + 15) & ~15;
            const float s0_scale = __ldg(a.s0_scale + req * a.s0_scale_req_stride + h);
            const float inv_s0 = 1.f / s0_scale;                            // a power of two
            if (n > MAXN || nd > MAXD || n < 1 || a.W > MAXW) {   // the host's choice of kernel was wrong for this input
                if (tb == 0 && atomicCAS(a.status, ONELA_OK, ONELA_E_UNSUPPORTED) == ONELA_OK) a.status[1] = n;
                give_up();
                break;
            }

            TL(10, seg);   // set-up start
            // ---------------- set-up of the segment ----------------
            // Keys and values of the distinct nodes: 16-byte async copies, neighbouring threads neighbouring chunks, every
            // copy of a thread in flight at once; a key chunk lands at its place in the operand tile as bf16 and is turned
            // into fp16 there by the thread that copied it (same size, same place).  A node's gates, level and ancestors
            // come from the byte-sized tables the index kernel left, every beam's chain nodes by 16-byte copies too.
            constexpr int CH_PER_THREAD = MAXN * 16 / 256;
            {
                const bool mine = tb < n;
                const int kappa = tb;
                int32_t nslot[CH_PER_THREAD];
#pragma unroll
                for (int it = 0; it < CH_PER_THREAD; ++it) {
                    const int ch = tb + 256 * it;
                    nslot[it] = ch < n * 16 ? __ldg(ulist + (ch >> 4)) : 0;
                }
                const int32_t slot = mine ? __ldg(ulist + kappa) : 0;
                uint4 ninfo = make_uint4(0u, 0u, 0u, 0u);
                if (mine) ninfo = __ldg(reinterpret_cast<const uint4*>(a.unode + (long long)req * (ONELA_UNODE_CAP * 16)) + kappa);
                if (seg == 0 || (pair - 1) / a.H != req) {       // (the same for all heads of the request)
                    const int cpr = (groups_per_pair * GN + 15) >> 4;     // 16-byte chunks per level
                    const uint8_t* src = a.sg8 + req * a.sg8_req_stride;
                    for (int idx = tb; idx < m * cpr; idx += 256) {
                        const int l = idx / cpr, c = idx - l * cpr;
                        cp_async16(smem_u32(&mi.sg[l][c * 16]), src + (long long)l * a.sg_stride + c * 16);
                    }
                }
#pragma unroll
                for (int it = 0; it < CH_PER_THREAD; ++it) {
                    const int ch = tb + 256 * it, kp = ch >> 4, c = ch & 15;
                    if (ch < n * 16) {
                        const char* src = kv + (plane_row0 + nslot[it]) * REC_BYTES + c * 16;
                        cp_async16(smem_u32(A_s + (c >> 3) * A_KB_STRIDE + (kp >> 3) * 1024 + (kp & 7) * 128 + (((c & 7) ^ (kp & 7)) << 4)), src);
                        cp_async16(smem_u32(VS_s + kp * (DV * 2) + c * 16), src + DK * 2);
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                TL(15, seg);
                if (mine) {
                    mi.gates[kappa] = __ldg(a.gates + plane_row0 + slot);
                    mi.lvl[kappa] = (uint8_t)(ninfo.z & 0xffu);
                    *reinterpret_cast<uint2*>(&mi.anc[kappa][0]) = make_uint2(ninfo.x, ninfo.y);
                }
            }
            for (int i = tb; i < MAXN * MAXL; i += 256) (&mi.ld[0][0])[i] = 0.f;
            TL(16, seg);
            TL(17, seg);
            if (seg >= 1) {     // S_0 of a later segment: every MMA of the previous one has completed (end of the loop)
                const float* row = a.s0 + req * a.s0_req_stride + (long long)h * (DV * DK) + (long long)row_i * DK;
#pragma unroll 1
                for (int kb = (bw >> 2) * 2; kb < (bw >> 2) * 2 + 2; ++kb) {
                    uint32_t v[16];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float4 x = __ldg(reinterpret_cast<const float4*>(row + kb * 32) + c);
                        v[2 * c] = pack_f16x2(x.x * s0_scale, x.y * s0_scale);
                        v[2 * c + 1] = pack_f16x2(x.z * s0_scale, x.w * s0_scale);
                    }
                    tmem_st16(tmem_base + S0_COL + kb * 16 + lane_bits, v);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            } else if (epi) {
                put_first_s0();
            }
            TL(18, seg);
            asm volatile("cp.async.wait_all;" ::: "memory");
            TL(19, seg);
#pragma unroll
            for (int it = 0; it < CH_PER_THREAD; ++it) {
                const int ch = tb + 256 * it, kp = ch >> 4, c = ch & 15;
                if (ch < n * 16) {
                    uint4* pk = reinterpret_cast<uint4*>(A_s + (c >> 3) * A_KB_STRIDE + (kp >> 3) * 1024 + (kp & 7) * 128 + (((c & 7) ^ (kp & 7)) << 4));
                    const uint4 x = *pk;
                    *pk = make_uint4(bf16x2_to_f16x2(x.x), bf16x2_to_f16x2(x.y), bf16x2_to_f16x2(x.z), bf16x2_to_f16x2(x.w));
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (!team_sync()) { give_up(); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            TL(11, seg);   // staged

            // S_0 K^T and the Gram block K K_deep^T, issued by one thread; meanwhile every node's decay product
            if (tb == 0) {
                bool ok = true;
                if (seg == 0) ok = wait_or_abort(bar_s0_first, 0, abort_flag);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (ok) {
                    const uint32_t idesc_p = idesc_f16(n16), idesc_d = idesc_f16(nd16);
                    const uint32_t abase = smem_u32(A_s);
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_f16_ts(tmem_base + PACC_COL, tmem_base + S0_COL + (kb * 4 + ks) * 8,
                                        umma_desc(abase + kb * A_KB_STRIDE + ks * 32), idesc_p, (kb | ks) ? 1u : 0u);
                    if (nd > 0) {
#pragma unroll
                        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                const uint64_t bd = umma_desc(abase + kb * A_KB_STRIDE + ks * 32);
                                umma_f16_ss(tmem_base + GRAM_LO_COL, bd, bd, idesc_d, (kb | ks) ? 1u : 0u);
                                if (n > 128)
                                    umma_f16_ss(tmem_base + GRAM_HI_COL, umma_desc(abase + HI_ROW0 * 128 + kb * A_KB_STRIDE + ks * 32), bd,
                                                idesc_d, (kb | ks) ? 1u : 0u);
                            }
                    }
                }
                umma_commit(bar_setup_mma);
                if (!ok) give_up();
            }
            if (tb < n) {
                const int kappa = tb, lv = mi.lvl[kappa];
                float e = mi.gates[kappa].x;
                for (int l = 0; l < lv; ++l) e *= mi.gates[mi.anc[kappa][l]].x;
                mi.ne[kappa] = e * inv_s0;
            }
            if (!warp_wait(bar_setup_mma, seg & 1, abort_flag)) give_up();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (!team_sync()) { give_up(); break; }
            TL(12, seg);   // set-up MMAs complete

            // U = [v_kappa - e_kappa S_0 k_kappa] into tensor memory as fp16 times one power of two: lane = output row,
            // the two teams take alternate blocks of 16 nodes.  The power of two comes from a bound on |u|, the largest
            // |v| plus the largest |e / scale| times the largest |S_0 k| (one cheap look at each), so U is written in
            // one pass.
            float u_scale = 1.f, u_inv = 1.f;
            {
                uint32_t vm = 0, pm = 0, nm = 0;
                for (int ch = tb; ch < n * 16; ch += 256) {
                    const uint4 w = *reinterpret_cast<const uint4*>(VS_s + ch * 16);
                    vm = __vmaxu2(vm, __vmaxu2(__vmaxu2(w.x & 0x7fff7fffu, w.y & 0x7fff7fffu), __vmaxu2(w.z & 0x7fff7fffu, w.w & 0x7fff7fffu)));
                }
                vm = max(vm & 0xffffu, vm >> 16) << 16;              // the largest bf16 magnitude, as fp32 bits
                TL(50, seg);
                for (int c0 = (bw >> 2) * 16; c0 < n16; c0 += 32) {
                    uint32_t pv[16];
                    tmem_ld16(tmem_base + PACC_COL + c0 + lane_bits, pv);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < n) pm = max(pm, pv[j] & 0x7fffffffu);
                }
                TL(51, seg);
                if (tb < n) nm = __float_as_uint(mi.ne[tb]) & 0x7fffffffu;
                vm = __reduce_max_sync(0xffffffffu, vm);
                pm = __reduce_max_sync(0xffffffffu, pm);
                nm = __reduce_max_sync(0xffffffffu, nm);
                if (lane == 0) {
                    mi.umax[bw] = vm;
                    mi.umax[8 + bw] = pm;
                    mi.umax[16 + bw] = nm;
                }
                if (!team_sync()) { give_up(); break; }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    vm = max(vm, mi.umax[i]);
                    pm = max(pm, mi.umax[8 + i]);
                    nm = max(nm, mi.umax[16 + i]);
                }
                TL(52, seg);
                pow2_scale(fmaf(__uint_as_float(nm), __uint_as_float(pm), __uint_as_float(vm)), U_TARGET, u_scale, u_inv);
                for (int c0 = (bw >> 2) * 16; c0 < n16; c0 += 32) {
                    uint32_t pv[16];
                    tmem_ld16(tmem_base + PACC_COL + c0 + lane_bits, pv);
                    // the nodes' factors and this row's value elements while the accumulator block is on its way
                    float vv[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int kappa = min(c0 + j, n - 1);
                        vv[j] = __uint_as_float((uint32_t)(*reinterpret_cast<const uint16_t*>(VS_s + kappa * (DV * 2) + row_i * 2)) << 16);
                    }
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    uint32_t w8[8];
#pragma unroll
                    for (int j = 0; j < 16; j += 2) {
                        const float u0 = c0 + j < n ? fmaf(-mi.ne[min(c0 + j, n - 1)], __uint_as_float(pv[j]), vv[j]) * u_scale : 0.f;
                        const float u1 = c0 + j + 1 < n ? fmaf(-mi.ne[min(c0 + j + 1, n - 1)], __uint_as_float(pv[j + 1]), vv[j + 1]) * u_scale : 0.f;
                        w8[j >> 1] = pack_f16x2(u0, u1);
                    }
                    tmem_st8(tmem_base + U_COL + (c0 >> 1) + lane_bits, w8);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            }
            TL(13, seg);   // U built
            // The chain dot products: a node's row of the Gram block goes through shared memory (as fp16, over the
            // second weight tile, idle now) so that the thread can pick its ancestors' columns.
            if (!epi && nd > 0) {
                for (int part_hi = 0; part_hi < ((n > 128 && quad == 2) ? 2 : 1); ++part_hi) {
                    const int kappa = part_hi ? 128 + lane : row_i;
                    uint8_t* bounce = slot_W(1) + row_i * 128;     // the thread's own 128 bytes (used twice by the third warp)
                    const uint32_t col = part_hi ? GRAM_HI_COL : GRAM_LO_COL;
                    for (int c0 = 0; c0 < nd16; c0 += 16) {
                        uint32_t p[16];
                        tmem_ld16(tmem_base + col + c0 + lane_bits, p);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        uint32_t w8[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) w8[j] = pack_f16x2(__uint_as_float(p[2 * j]), __uint_as_float(p[2 * j + 1]));
                        *reinterpret_cast<uint4*>(bounce + c0 * 2) = make_uint4(w8[0], w8[1], w8[2], w8[3]);
                        *reinterpret_cast<uint4*>(bounce + c0 * 2 + 16) = make_uint4(w8[4], w8[5], w8[6], w8[7]);
                    }
                    __syncwarp();
                    if (kappa < n) {
                        const int lv = mi.lvl[kappa];
                        for (int l = 0; l < lv; ++l)
                            mi.ld[kappa][l] = __half2float(*reinterpret_cast<const __half*>(bounce + mi.anc[kappa][l] * 2));
                    }
                    __syncwarp();
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (!team_sync()) { give_up(); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

            TL(14, seg);   // set-up done
            // ---------------- the segment's groups ----------------
            if (epi) {
                const int te = tid - EPI_WARP0 * 32;          // 0 .. 127
                float* T_s = reinterpret_cast<float*>(T_raw);
                dependency_wait();
                for (int gi = seg_g0; gi < seg_g1; ++gi, ++gcount) {
                    const int s = gcount % SLOTS, vs = gcount % VSLOTS;
                    const int b0 = (gi - pair * groups_per_pair) * GN;
                    TL(20, gcount);   // epilogue: waiting for U . W^T
                    if (!fail && !warp_wait(bar_done2(s), (gcount / SLOTS) & 1, abort_flag)) give_up();
                    TL(21, gcount);   // epilogue: accumulators complete
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (!fail) {
                        const int ip = corr_chunk(row_i >> 2) * 4 + (row_i & 3);
#pragma unroll
                        for (int c0 = 0; c0 < GN; c0 += 16) {
                            uint32_t x1[16], x2[16];
                            tmem_ld16(tmem_base + ACC1_COL + vs * GN + c0 + lane_bits, x1);
                            tmem_ld16(tmem_base + ACC2_COL + s * GN + c0 + lane_bits, x2);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                            for (int j4 = 0; j4 < 16; j4 += 4) {
                                const float4 ca = *reinterpret_cast<const float4*>(&mi.cA[vs][c0 + j4]);
                                const float4 cb = *reinterpret_cast<const float4*>(&mi.cB[vs][c0 + j4]);
                                T_s[(c0 + j4 + 0) * DV + ip] = fmaf(ca.x, __uint_as_float(x1[j4 + 0]), cb.x * __uint_as_float(x2[j4 + 0]));
                                T_s[(c0 + j4 + 1) * DV + ip] = fmaf(ca.y, __uint_as_float(x1[j4 + 1]), cb.y * __uint_as_float(x2[j4 + 1]));
                                T_s[(c0 + j4 + 2) * DV + ip] = fmaf(ca.z, __uint_as_float(x1[j4 + 2]), cb.z * __uint_as_float(x2[j4 + 2]));
                                T_s[(c0 + j4 + 3) * DV + ip] = fmaf(ca.w, __uint_as_float(x1[j4 + 3]), cb.w * __uint_as_float(x2[j4 + 3]));
                            }
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    if (bar_or(1, 128, fail ? 1 : 0)) { dead = true; break; }
                    TL(22, gcount);   // epilogue: tile transposed
                    {
                        OutT* out0 = static_cast<OutT*>(a.out) + (((long long)req * a.W + b0) * a.H + h) * DV;
                        const uint8_t* V_s = slot_V(vs);
#pragma unroll
                        for (int it = 0; it < GN * 16 / 128; ++it) {
                            const int idx = it * 128 + te, j = idx >> 4, ch = idx & 15;
                            if (b0 + j < a.W) {
                                const float4 y0 = *reinterpret_cast<const float4*>(T_s + j * DV + corr_chunk(2 * ch) * 4);
                                const float4 y1 = *reinterpret_cast<const float4*>(T_s + j * DV + corr_chunk(2 * ch + 1) * 4);
                                const uint4 vv = *reinterpret_cast<const uint4*>(V_s + j * (DV * 2) + ch * 16);
                                float2 vx[4];
                                unpack8(vv, vx);
                                const float w = mi.wt[vs][j];
                                const float o[8] = {fmaf(vx[0].x, w, y0.x), fmaf(vx[0].y, w, y0.y), fmaf(vx[1].x, w, y0.z), fmaf(vx[1].y, w, y0.w),
                                                    fmaf(vx[2].x, w, y1.x), fmaf(vx[2].y, w, y1.y), fmaf(vx[3].x, w, y1.z), fmaf(vx[3].y, w, y1.w)};
                                store8<OutT>(out0 + (long long)j * a.H * DV + ch * 8, o);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_free(vs));
                    named_bar(1, 128);      // the transposed tile is read out before the next group's goes in
                    TL(23, gcount);   // epilogue: group done
                }
            } else {
                const int ts = tid - SOL_WARP0 * 32;          // 0 .. 127
                const int my_lvl = row_i < n ? mi.lvl[row_i] : -1;
                const int hi_kappa = 128 + lane;
                const int hi_lvl = (quad == 2 && hi_kappa < n) ? mi.lvl[hi_kappa] : -1;
                // [S_0 ; K] . R^T of group gc, by the first lane of the last solver warp (which has no beam to solve for);
                // true: gave up.  K . R^T has one buffer: the caller has seen the previous group's read out.
                auto issue_mma1 = [&](int gc) -> bool {
                    const int s = gc % SLOTS, vs = gc % VSLOTS;
                    int failed = 0;
                    if (lane == 0) {
                        TL(40, gc);   // issue: waiting for the fold warps
                        const bool ok = wait_or_abort(bar_full(s), (gc / SLOTS) & 1, abort_flag);
                        TL(41, gc);   // issue: rows complete
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        if (ok) {
                            const uint32_t rbase = smem_u32(slot_R(s)), abase = smem_u32(A_s);
#pragma unroll
                            for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                                for (int ks = 0; ks < 4; ++ks) {
                                    const uint64_t bd = umma_desc(rbase + kb * R_KB_STRIDE + ks * 32);
                                    const uint32_t acc = (kb | ks) ? 1u : 0u;
                                    umma_f16_ss(tmem_base + GLO_COL, umma_desc(abase + kb * A_KB_STRIDE + ks * 32), bd, idesc_g, acc);
                                    if (n > 128)
                                        umma_f16_ss(tmem_base + GHI_COL, umma_desc(abase + HI_ROW0 * 128 + kb * A_KB_STRIDE + ks * 32), bd, idesc_g, acc);
                                    umma_f16_ts(tmem_base + ACC1_COL + vs * GN, tmem_base + S0_COL + (kb * 4 + ks) * 8, bd, idesc_g, acc);
                                }
                        } else {
                            failed = 1;
                        }
                        umma_commit(bar_done1(s));
                        TL(42, gc);   // issue: MMAs out
                    }
                    return __shfl_sync(0xffffffffu, failed, 0) != 0;
                };
                if (warp == ISS_WARP && issue_mma1(gcount)) give_up();      // the segment's first group
                for (int gi = seg_g0; gi < seg_g1; ++gi, ++gcount) {
                    const int s = gcount % SLOTS, vs = gcount % VSLOTS;
                    const int b0 = (gi - pair * groups_per_pair) * GN;
                    TL(30, gcount);   // solver: waiting for K . R^T
                    if (!fail && !warp_wait(bar_done1(s), (gcount / SLOTS) & 1, abort_flag)) give_up();
                    // the weight tile is free once the U . W^T of group gcount - 2 has completed
                    if (!fail && gcount >= SLOTS && !warp_wait(bar_done2(s), ((gcount / SLOTS) - 1) & 1, abort_flag)) give_up();
                    TL(31, gcount);   // solver: K . R^T complete
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    if (!fail) {
                        // lane = node: hand each beam of the group the entry of its chain's node at this node's level
                        uint32_t x[GN];
#pragma unroll
                        for (int c0 = 0; c0 < GN; c0 += 16) tmem_ld16(tmem_base + GLO_COL + c0 + lane_bits, x + c0);
                        // the weight tile starts from zero
                        uint4* wz = reinterpret_cast<uint4*>(slot_W(s));
#pragma unroll
                        for (int i = 0; i < W_BYTES / 16 / 128; ++i) wz[i * 128 + ts] = make_uint4(0u, 0u, 0u, 0u);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if (my_lvl >= 0) {
                            const uint32_t me = (uint32_t)row_i * 0x01010101u;
                            const uint32_t* ids = reinterpret_cast<const uint32_t*>(&mi.sg[my_lvl][b0]);
#pragma unroll
                            for (int q4 = 0; q4 < GN / 4; ++q4) {
                                const uint32_t eq = __vcmpeq4(ids[q4], me);
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    if (eq & (0xffu << (8 * j))) mi.gout[s][my_lvl][q4 * 4 + j] = __uint_as_float(x[q4 * 4 + j]);
                            }
                        }
                        if (n > 128 && quad == 2) {
#pragma unroll
                            for (int c0 = 0; c0 < GN; c0 += 16) tmem_ld16(tmem_base + GHI_COL + c0 + lane_bits, x + c0);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                            if (hi_lvl >= 0) {
                                const uint32_t me = (uint32_t)hi_kappa * 0x01010101u;
                                const uint32_t* ids = reinterpret_cast<const uint32_t*>(&mi.sg[hi_lvl][b0]);
#pragma unroll
                                for (int q4 = 0; q4 < GN / 4; ++q4) {
                                    const uint32_t eq = __vcmpeq4(ids[q4], me);
#pragma unroll
                                    for (int j = 0; j < 4; ++j)
                                        if (eq & (0xffu << (8 * j))) mi.gout[s][hi_lvl][q4 * 4 + j] = __uint_as_float(x[q4 * 4 + j]);
                                }
                            }
                        }
                    }
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    if (bar_or(2, 128, fail ? 1 : 0)) { dead = true; break; }
                    TL(32, gcount);   // solver: entries handed out
                    if (warp == ISS_WARP) {
                        // K . R^T has been read out: the next group's MMAs go out while the first two warps solve
                        if (gi + 1 < seg_g1 && issue_mma1(gcount + 1)) give_up();     // (carried to the next group's barrier)
                        continue;
                    }
                    if (warp >= SOL_WARP0 + 2) continue;      // the third warp has no beams either
                    if (ts < GN) {
                        // one beam per thread: the triangular solve along its chain, newest of the older levels first
                        const int u = ts;
                        const float f = mi.fA[vs][u];
                        // Levels beyond the chain read the parent's entries and count for nothing (their beta is taken as 0).
                        // A solved level is taken out of all older levels' right-hand sides at once: its row of chain dot
                        // products is contiguous (two 16-byte loads).
                        int kap[MAXL];
#pragma unroll
                        for (int l = 0; l < MAXL; ++l) kap[l] = mi.sg[min(l, m - 1)][b0 + u];
                        float2 gt[MAXL];
                        float gg[MAXL], w[MAXL];
#pragma unroll
                        for (int l = 0; l < MAXL; ++l) {
                            const float2 gl = mi.gates[kap[l]];
                            const float go = mi.gout[s][min(l, m - 1)][u];
                            gt[l] = l < m ? gl : make_float2(1.f, 0.f);
                            gg[l] = l < m ? go : 0.f;
                        }
                        TL(35, gcount);
                        float d = 1.f, wmax = 0.f;
#pragma unroll
                        for (int l = MAXL - 1; l >= 0; --l) {
                            const float bc = gt[l].y * gg[l];
                            w[l] = bc * d * f;
                            wmax = fmaxf(wmax, fabsf(w[l]));
                            d *= gt[l].x;
                            if (l > 0) {
                                const float4 r0 = *reinterpret_cast<const float4*>(&mi.ld[kap[l]][0]);
                                gg[0] = fmaf(-bc, r0.x, gg[0]);
                                if (l > 1) gg[1] = fmaf(-bc, r0.y, gg[1]);
                                if (l > 2) gg[2] = fmaf(-bc, r0.z, gg[2]);
                                if (l > 3) gg[3] = fmaf(-bc, r0.w, gg[3]);
                                if (l > 4) {
                                    const float4 r1 = *reinterpret_cast<const float4*>(&mi.ld[kap[l]][4]);
                                    gg[4] = fmaf(-bc, r1.x, gg[4]);
                                    if (l > 5) gg[5] = fmaf(-bc, r1.y, gg[5]);
                                    if (l > 6) gg[6] = fmaf(-bc, r1.z, gg[6]);
                                }
                            }
                        }
                        TL(36, gcount);
                        float w_scale, w_inv;
                        pow2_scale(wmax, W_TARGET, w_scale, w_inv);
                        mi.cA[vs][u] = d * f * inv_s0;
                        mi.cB[vs][u] = w_inv * u_inv;
                        uint8_t* wrow = slot_W(s) + (u >> 3) * 1024 + (u & 7) * 128;
#pragma unroll
                        for (int l = 0; l < MAXL; ++l)
                            if (l < m) {
                                const int kp = kap[l];
                                *reinterpret_cast<__half*>(wrow + (kp >> 6) * W_KB_STRIDE + ((((kp & 63) >> 3) ^ (u & 7)) << 4) + (kp & 7) * 2) =
                                    __float2half_rn(w[l] * w_scale);
                            }
                    }
                    TL(37, gcount);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    TL(33, gcount);   // solver: solved
                    named_bar(3, 64);       // the two solving warps
                    TL(38, gcount);
                    if (ts == 0) {
                        // the accumulator is free once the epilogue of group gcount - 2 has read it
                        bool ok = true;
                        if (gcount >= SLOTS) ok = wait_or_abort(bar_free((gcount - SLOTS) % VSLOTS), ((gcount - SLOTS) / VSLOTS) & 1, abort_flag);
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        if (ok) {
                            const uint32_t wbase = smem_u32(slot_W(s));
                            for (int kk = 0; kk < n16 / 16; ++kk)
                                umma_f16_ts(tmem_base + ACC2_COL + s * GN, tmem_base + U_COL + kk * 8,
                                            umma_desc(wbase + (kk >> 2) * W_KB_STRIDE + (kk & 3) * 32), idesc_g, kk ? 1u : 0u);
                        } else {
                            *abort_flag = 1;
                        }
                        umma_commit(bar_done2(s));
                    }
                    TL(34, gcount);   // solver: U . W^T issued
                }
            }
            if (dead) break;
            // before the next segment's set-up overwrites S_0, U and the key tile, both teams have finished this one
            if (seg + 1 < n_segs) {
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                if (!team_sync()) { give_up(); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            }
        }
        if (fail) dead = true;
    }
    if (dead && lane == 0) {
        *abort_flag = 1;
        if (atomicCAS(a.status, ONELA_OK, ONELA_E_TIMEOUT) == ONELA_OK) a.status[1] = (int32_t)blockIdx.x;
    }
#ifdef ONELA_WY_TL
    if (lane == 0 && tl_role >= 0) {
        for (int i = 0; i < tl_n; ++i) g_wy_tl[tl_role * TL_CAP + i] = tl_s[tl_role * TL_CAP + i];
        g_wy_tl_n[tl_role] = tl_n;
    }
#endif
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <typename OutT, bool FUSED>
cudaError_t launch_wy_t(const DecodeArgs& a, cudaStream_t stream) {
    auto kern = decode_wy_kernel<OutT, FUSED>;
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
            const int n = decode_sm_count();
            sms_of[dev] = n > DECODE_MAX_CTAS ? DECODE_MAX_CTAS : n;
        }
        sms = sms_of[dev];
    }
    const int groups_per_pair = (a.W + GN - 1) / GN;
    const int total_groups = a.req_count * a.H * groups_per_pair;
    // Starting a segment costs about as much as three groups here (the tables are rebuilt), so a CTA keeps whole
    // (request, head) pairs where there are enough of them.
    static thread_local DecodePartition part;
    static thread_local int part_total = -1, part_gpp = -1, part_sms = -1, part_ctas = 0;
    if (part_total != total_groups || part_gpp != groups_per_pair || part_sms != sms) {
        part_ctas = make_decode_partition(total_groups, groups_per_pair, sms, 8, 24, &part);
        part_total = total_groups; part_gpp = groups_per_pair; part_sms = sms;
    }
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

#ifdef ONELA_WY_TL
extern "C" int onela_debug_wy_timeline(unsigned long long* out_host, int* counts_host) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(counts_host, g_wy_tl_n, 4 * sizeof(int));
    cudaMemcpyFromSymbol(out_host, g_wy_tl, sizeof(unsigned long long) * 4 * TL_CAP);
    const int zero[4] = {0, 0, 0, 0};
    cudaMemcpyToSymbol(g_wy_tl_n, zero, sizeof(zero));
    return TL_CAP;
}
#endif

cudaError_t launch_decode_wy(const DecodeArgs& a, int32_t out_dtype, cudaStream_t stream) {
    const bool fused = a.k_in != nullptr;
    const bool bf16 = out_dtype == ONELA_DTYPE_BF16;
    if (fused) return bf16 ? launch_wy_t<__nv_bfloat16, true>(a, stream) : launch_wy_t<float, true>(a, stream);
    return bf16 ? launch_wy_t<__nv_bfloat16, false>(a, stream) : launch_wy_t<float, false>(a, stream);
}

}  // namespace onela
