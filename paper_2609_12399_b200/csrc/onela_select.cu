// Global beam selection (Section 2.1: every active beam is expanded over the codebook and the global top-k
// candidates are kept): from the previous beams' cumulative scores and this step's candidate log-probabilities,
// the W_new best (parent, code) pairs per request, best first, parents in the form onela_reorder_beams takes - so
// selection, reorder and the layers' decode launches of a step can run back to back on the device (one CUDA graph).
//
// A candidate's rank is a 64-bit composite: its fp32 score (parent score + log-probability, mapped to
// order-preserving bits; NaN lowest, -0 = +0) in the high word, 0xffffffff - flat index in the low word, so
// composites are distinct and "larger" means "better, ties to the smaller flat index".  A CTA finds the k largest
// composites of a range by an 8-bit radix select from the top byte down (the passes over the index bytes are
// skipped when no tie straddles the cut) and gathers them in shared memory.
// Two launches per call: `select_part_kernel` cuts a request's candidates into parts of 4096 and leaves each part's
// own top-k (unordered) in a scratch area of the workspace; `select_merge_kernel` (one CTA per request) selects
// among those and orders the survivors with a bitonic sort.  A request with a single part skips the scratch.
#include <mutex>

#include "onela_internal.h"

namespace onela {

namespace {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_CAP = ONELA_SELECT_CAP;      // survivors per request (W_new <= SEL_CAP)
constexpr int SEL_PART = 4096;                 // candidates per part: four per thread
constexpr int SEL_PARTS_MAX = ONELA_SELECT_PARTS;

__device__ __forceinline__ uint32_t score_bits(float s) {
    if (s != s) return 0u;                              // NaN: below every number
    const uint32_t u = __float_as_uint(s + 0.0f);       // -0.0 + 0.0 = +0.0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct ScoreSource {     // composites computed from the caller's scores; item i is flat index first + i
    const float* bs;
    const float* lp;
    uint32_t first;
    int C;
    __device__ __forceinline__ unsigned long long operator()(uint32_t i) const {
        const uint32_t idx = first + i;
        const float s = __ldg(bs + idx / (uint32_t)C) + __ldg(lp + idx);
        return ((unsigned long long)score_bits(s) << 32) | (unsigned long long)(0xffffffffu - idx);
    }
};
struct SelectShared {
    unsigned int hist[256];
    unsigned long long sel[SEL_CAP];
    unsigned long long prefix;
    unsigned int k, count, equal;
};

// Leaves the k largest composites of item(0 .. n-1) in sh.sel[0 .. k) (unordered); k <= min(n, SEL_CAP).
// `item(j, i)` returns composite i = tid + j * SEL_THREADS: from the source itself, or from the thread's registers.
// MAXJ > 0: at most MAXJ items per thread, loops unrolled (so that a register array can be indexed); 0: any number.
template <int MAXJ, class Item>
__device__ void select_passes(const Item& item, uint32_t n, int k, SelectShared& sh) {
    const int tid = threadIdx.x;
    if (tid == 0) { sh.prefix = 0ull; sh.k = (unsigned)k; sh.count = 0u; }
    if (tid < 256) sh.hist[tid] = 0u;
    __syncthreads();
    // after the pass over byte p, sh.prefix holds bytes 7..p of the k-th largest composite and sh.k how many
    // survivors are still to be found among the candidates that share those bytes
    const uint32_t n_padded = (n + SEL_THREADS - 1) / SEL_THREADS * SEL_THREADS;
    for (int p = 7; p >= 0; --p) {             // two block-wide barriers per pass
        const unsigned long long prefix = sh.prefix;
        const unsigned want = sh.k;               // (read here: the bin search below rewrites it)
        const unsigned long long hi_mask = p == 7 ? 0ull : (~0ull << (8 * (p + 1)));
        auto count_item = [&](int j, uint32_t i) {
            // whole warps stay in the loop (padding iterations carry no candidate) so the peer vote is complete
            const bool live = i < n;
            const unsigned long long c = live ? item(j, i) : 0ull;
            const bool in = live && ((c & hi_mask) == prefix);
            const unsigned bin = (unsigned)(c >> (8 * p)) & 255u;
            // one atomic per distinct bin in the warp: scores cluster, so most lanes share a bin in the early passes
            const unsigned vote = __ballot_sync(0xffffffffu, in);
            if (in) {
                const unsigned peers = __match_any_sync(vote, bin);
                if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&sh.hist[bin], __popc(peers));
            }
        };
        if constexpr (MAXJ > 0) {
#pragma unroll
            for (int j = 0; j < MAXJ; ++j) {
                const uint32_t i = tid + (uint32_t)j * SEL_THREADS;
                if (i < n_padded) count_item(j, i);
            }
        } else {
            for (uint32_t i = tid; i < n_padded; i += SEL_THREADS) count_item(0, i);
        }
        __syncthreads();
        // the bin that holds the k-th largest, by the first warp alone: lane l takes bins 8 l .. 8 l + 7, suffix counts
        // (candidates in bins >= b) across the lanes by shuffles; it also clears the histogram for the next pass
        if (tid < 32) {
            unsigned h[8], mine = 0;
#pragma unroll
            for (int t = 0; t < 8; ++t) { h[t] = sh.hist[8 * tid + t]; mine += h[t]; }
#pragma unroll
            for (int t = 0; t < 8; ++t) sh.hist[8 * tid + t] = 0u;
            unsigned incl = mine;                                   // counts of lanes >= this one
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned up = __shfl_down_sync(0xffffffffu, incl, off);
                if (tid + off < 32) incl += up;
            }
            unsigned here = incl;                                   // candidates in bins >= 8 tid + t, from t = 0 down
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const unsigned next = here - h[t];                  // ... in bins > 8 tid + t
                if (here >= want && next < want) {                  // exactly one bin qualifies
                    sh.prefix = prefix | ((unsigned long long)(8 * tid + t) << (8 * p));
                    sh.k = want - next;
                    sh.equal = h[t];
                }
                here = next;
            }
        }
        __syncthreads();
        // the score word is fixed and exactly the candidates that share it are still wanted: no tie straddles the cut
        if (p == 4 && sh.equal == sh.k) break;
    }
    const unsigned long long threshold = sh.prefix;   // (low bytes zero after an early exit: every equal score is kept)
    auto keep_item = [&](int j, uint32_t i) {
        const unsigned long long c = item(j, i);
        if (c >= threshold) {
            const unsigned pos = atomicAdd(&sh.count, 1u);
            if (pos < SEL_CAP) sh.sel[pos] = c;
        }
    };
    if constexpr (MAXJ > 0) {
#pragma unroll
        for (int j = 0; j < MAXJ; ++j) {
            const uint32_t i = tid + (uint32_t)j * SEL_THREADS;
            if (i < n) keep_item(j, i);
        }
    } else {
        for (uint32_t i = tid; i < n; i += SEL_THREADS) keep_item(0, i);
    }
    __syncthreads();
}
// The passes read every candidate four to eight times.  Up to ITEMS * SEL_THREADS candidates are fetched once, all
// loads in flight together, and kept in registers (a pass then costs votes and shared-memory atomics only: the
// merging CTA fell from 48 us to a fraction of that on 16 384 composites); longer lists are re-read from the source.
template <int ITEMS, class Src>
__device__ void select_topk(const Src& src, uint32_t n, int k, SelectShared& sh) {
    if (n <= (uint32_t)ITEMS * SEL_THREADS) {
        unsigned long long held[ITEMS];
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            const uint32_t i = threadIdx.x + (uint32_t)j * SEL_THREADS;
            held[j] = i < n ? src(i) : 0ull;
        }
        auto item = [&](int j, uint32_t) { return held[j]; };      // j is a compile-time constant in the unrolled loops
        select_passes<ITEMS>(item, n, k, sh);
    } else {
        auto item = [&](int, uint32_t i) { return src(i); };
        select_passes<0>(item, n, k, sh);
    }
}

// Orders sh.sel[0 .. k) best first and writes the survivors out.
__device__ void sort_and_emit(SelectShared& sh, int k, const float* bs, const float* lp, int C, int32_t* parents,
                              int32_t* codes, float* scores) {
    const int tid = threadIdx.x;
    int n_sort = 2;
    while (n_sort < k) n_sort <<= 1;                        // the sort runs over the next power of two
    for (int i = tid; i < n_sort; i += SEL_THREADS)
        if (i >= k) sh.sel[i] = 0ull;
    __syncthreads();
    // Bitonic sort, descending.  Compare-exchange i of a step pairs elements inside the 64-element block i / 32 whenever
    // the stride is below 64, and thread i (= pair i; n_sort / 2 <= 512 pairs) belongs to warp i / 32: those steps need
    // the warp only, and a block-wide barrier stands just before and after each run of them.
    auto exchange = [&](int i, int size, int stride) {
        const int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
        const bool desc = (lo & size) == 0;
        const unsigned long long x = sh.sel[lo], y = sh.sel[hi];
        if ((x < y) == desc) { sh.sel[lo] = y; sh.sel[hi] = x; }
    };
    static_assert(SEL_CAP / 2 <= SEL_THREADS, "one compare-exchange per thread and step");
    const bool mine = tid < n_sort / 2;
    for (int size = 2; size <= n_sort; size <<= 1) {
        int stride = size >> 1;
        for (; stride >= 64; stride >>= 1) {                // partners in different 64-element blocks
            if (mine) exchange(tid, size, stride);
            __syncthreads();
        }
        for (; stride > 0; stride >>= 1) {                  // partners inside this warp's 64-element block
            if (mine) exchange(tid, size, stride);
            __syncwarp();
        }
        __syncthreads();
    }
    for (int i = tid; i < k; i += SEL_THREADS) {
        const uint32_t idx = 0xffffffffu - (uint32_t)(sh.sel[i] & 0xffffffffull);
        const int par = (int)(idx / (uint32_t)C);
        parents[i] = par;
        codes[i] = (int)(idx - (uint32_t)par * (uint32_t)C);
        scores[i] = __ldg(bs + par) + __ldg(lp + idx);
    }
}

// grid (parts, requests): the part's own top-k, unordered, to scratch[request][part][0 .. kp), kp = min(k, part size)
__global__ void __launch_bounds__(SEL_THREADS) select_part_kernel(const float* __restrict__ beam_scores, const float* __restrict__ cand_logp,
                                                                  int W_prev, int C, int k, unsigned long long* __restrict__ scratch) {
    __shared__ SelectShared sh;
    const int part = blockIdx.x, req = blockIdx.y;
    const uint32_t N = (uint32_t)W_prev * (uint32_t)C, first = (uint32_t)part * SEL_PART;
    const uint32_t n = min((uint32_t)SEL_PART, N - first);
    const int kp = min((uint32_t)k, n);
    const ScoreSource src{beam_scores + (long long)req * W_prev, cand_logp + (long long)req * W_prev * C, first, C};
    select_topk<SEL_PART / SEL_THREADS>(src, n, kp, sh);
    unsigned long long* out = scratch + ((long long)req * SEL_PARTS_MAX + part) * SEL_CAP;
    for (int i = threadIdx.x; i < kp; i += SEL_THREADS) out[i] = sh.sel[i];
}

// one CTA per request: the top-k of the parts' lists (parts > 1) or of the candidates themselves (parts == 1)
__global__ void __launch_bounds__(SEL_THREADS) select_merge_kernel(const float* __restrict__ beam_scores, const float* __restrict__ cand_logp,
                                                                   int W_prev, int C, int k, int parts,
                                                                   const unsigned long long* __restrict__ scratch, int32_t* __restrict__ parents,
                                                                   int32_t* __restrict__ codes, float* __restrict__ scores) {
    __shared__ SelectShared sh;
    const int req = blockIdx.x;
    const float* bs = beam_scores + (long long)req * W_prev;
    const float* lp = cand_logp + (long long)req * W_prev * C;
    const uint32_t N = (uint32_t)W_prev * (uint32_t)C;
    if (parts == 1) {
        select_topk<SEL_PART / SEL_THREADS>(ScoreSource{bs, lp, 0u, C}, N, k, sh);
    } else {
        // every part but the last left min(k, SEL_PART) composites; read them as one list with gaps skipped
        const uint32_t kp = min((uint32_t)k, (uint32_t)SEL_PART);
        const uint32_t last_n = N - (uint32_t)(parts - 1) * SEL_PART, last_kp = min((uint32_t)k, last_n);
        struct Gapped {
            const unsigned long long* base;
            uint32_t kp;
            __device__ __forceinline__ unsigned long long operator()(uint32_t i) const {
                return base[(long long)(i / kp) * SEL_CAP + (i % kp)];
            }
        };
        const Gapped src{scratch + (long long)req * SEL_PARTS_MAX * SEL_CAP, kp};
        select_topk<16>(src, (uint32_t)(parts - 1) * kp + last_kp, k, sh);
    }
    sort_and_emit(sh, k, bs, lp, C, parents + (long long)req * k, codes + (long long)req * k, scores + (long long)req * k);
}

}  // namespace

cudaError_t launch_select(const float* beam_scores, const float* cand_logp, int32_t req_count, int32_t W_prev, int32_t C,
                          int32_t W_new, unsigned long long* scratch, int32_t* parents, int32_t* codes, float* scores,
                          cudaStream_t stream) {
    const long long N = (long long)W_prev * C;
    const int parts = (int)((N + SEL_PART - 1) / SEL_PART);
    if (parts > SEL_PARTS_MAX) return cudaErrorInvalidValue;
    if (parts > 1) {
        select_part_kernel<<<dim3(parts, req_count), SEL_THREADS, 0, stream>>>(beam_scores, cand_logp, W_prev, C, W_new, scratch);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    select_merge_kernel<<<req_count, SEL_THREADS, 0, stream>>>(beam_scores, cand_logp, W_prev, C, W_new, parts, scratch, parents,
                                                               codes, scores);
    return cudaGetLastError();
}

}  // namespace onela

// ---------------------------------------------------------------------------------------------------------------
// Beam selection without a workspace (declared in onela.h as onela_select_beams_static).
//
// The partial lists go to an array that is part of the library image instead of the caller's workspace.  Its size is
// fixed when the library is built: room for STATIC_REQUESTS requests of the same candidate count the workspace
// version takes (ONELA_SELECT_PARTS parts of 4096 candidates, ONELA_SELECT_CAP survivors each) = 4 MiB, which
// every GPU that loads the library holds until the process ends.  In host code the array's name is only a handle;
// the device address comes from cudaGetSymbolAddress, asked for once per device on that device's first call.
namespace onela {
namespace {

constexpr int STATIC_REQUESTS = 2;
static __device__ __align__(256) unsigned long long g_static_select_scratch[(size_t)STATIC_REQUESTS * ONELA_SELECT_PARTS * ONELA_SELECT_CAP];

constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
unsigned long long* g_static_ptr[MAX_DEVICES] = {};

// device address of the array on the current device; nullptr when the runtime refuses
unsigned long long* static_scratch_of_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_select_scratch) != cudaSuccess) return nullptr;
        g_static_ptr[dev] = static_cast<unsigned long long*>(p);
    }
    return g_static_ptr[dev];
}

}  // namespace
}  // namespace onela

extern "C" onela_status onela_select_beams_static(const float* beam_scores_dev, const float* cand_logp_dev, int32_t req_count,
                                                  int32_t W_prev, int32_t C, int32_t W_new, int32_t* parents_out_dev,
                                                  int32_t* codes_out_dev, float* scores_out_dev, void* stream) {
    using namespace onela;
    if (!beam_scores_dev || !cand_logp_dev || !parents_out_dev || !codes_out_dev || !scores_out_dev) return ONELA_E_INVAL;
    if (req_count < 1 || W_prev < 1 || C < 1 || W_new < 1) return ONELA_E_INVAL;
    // beyond what the built-in array holds: the caller has to use onela_select_beams with a workspace, or split the batch
    if (req_count > STATIC_REQUESTS) return ONELA_E_CAPACITY;
    if ((int64_t)W_prev * C > (int64_t)ONELA_SELECT_PARTS * 4096) return ONELA_E_CAPACITY;
    if (W_new > ONELA_SELECT_CAP || W_new > (int64_t)W_prev * C) return ONELA_E_CAPACITY;
    unsigned long long* scratch = static_scratch_of_current_device();
    if (!scratch) return ONELA_E_CUDA;
    // nothing in the array has to start at zero: every word the merge step reads is written by the part step of
    // the same call
    if (launch_select(beam_scores_dev, cand_logp_dev, req_count, W_prev, C, W_new, scratch, parents_out_dev, codes_out_dev,
                      scores_out_dev, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return ONELA_E_CUDA;
    return ONELA_OK;
}
