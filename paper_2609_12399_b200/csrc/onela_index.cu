// Ancestry index kernels (paper Section 3.3, Eq. 5).  Integer work only: beam selection prunes,
// reorders and fans out beams by rewriting slot ids; no transition record is moved or copied.
//
// Table layout per request: two buffers [max_steps][max_beam] of int32 global slot ids, level-major
// (row `level` holds, for every live beam, the slot of its ancestor's record written at decode call
// `level`; the last live row is the beam's own record).  Buffer (depth-1)&1 is current at depth `depth`.
#include "onela_internal.h"

namespace onela {

namespace {

__global__ void __launch_bounds__(256) reorder_kernel(int32_t* __restrict__ tables_req0, long long table_req_stride,
                                                      const int32_t* __restrict__ parents, int32_t W_new,
                                                      int32_t W_prev, int32_t depth_old, int32_t max_beam,
                                                      int32_t max_steps, BatchBases bases,
                                                      int32_t* __restrict__ status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    const int level = blockIdx.y;   // 0 .. depth_old
    const int r = blockIdx.z;       // request within the batch
    if (b >= W_new) return;
    int32_t* tab = tables_req0 + r * table_req_stride;
    const long long buf = (long long)max_steps * max_beam;
    int32_t* newt = tab + (depth_old & 1) * buf;
    if (level == depth_old) {
        // h_t(b, t) : the record this beam is about to append lives at base(req, t) + b
        newt[(long long)level * max_beam + b] = bases.base[r] + b;
        return;
    }
    // Eq. 5: the child inherits its parent's row (levels < t-1) and, at level t-1, the parent's own
    // slot, which is the last entry of the parent's row - one gather covers both cases.
    const int32_t* oldt = tab + ((depth_old - 1) & 1) * buf;
    int p = parents[(long long)r * W_new + b];
    if ((unsigned)p >= (unsigned)W_prev) {
        if (atomicCAS(status, ONELA_OK, ONELA_E_DEVICE_CHECK) == ONELA_OK) status[1] = p;
        p = 0;
    }
    newt[(long long)level * max_beam + b] = oldt[(long long)level * max_beam + p];
}

__global__ void __launch_bounds__(256) export_chains_kernel(const int32_t* __restrict__ table, int32_t W, int32_t depth,
                                                            int32_t max_beam, int32_t* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= W * depth) return;
    const int b = i / depth, level = i % depth;
    out[i] = table[(long long)level * max_beam + b];
}

// One CTA per request.  For every level older than the beams' own records: mark which slots of that
// level some live chain refers to (slots of one level of one request are consecutive, so slot - min is a
// dense key < max_beam), prefix-sum the marks, and emit the distinct slots in increasing order plus each
// beam's position in the request's concatenated list, and for every distinct slot one beam that refers to it.
__global__ void __launch_bounds__(1024) dedupe_kernel(const int32_t* __restrict__ tables_cur_req0, long long table_req_stride,
                                                      int32_t* __restrict__ sidx_req0, long long sidx_req_stride,
                                                      int32_t* __restrict__ ulist_req0, long long ulist_req_stride,
                                                      int32_t* __restrict__ urep_req0,
                                                      int32_t* __restrict__ uoff_req0, long long uoff_req_stride,
                                                      uint8_t* __restrict__ sg8_req0, long long sg8_req_stride, int32_t sg_stride,
                                                      uint8_t* __restrict__ unode_req0,
                                                      int32_t W, int32_t depth, int32_t max_beam) {
    extern __shared__ int32_t marks[];          // [max_beam] marks, then their exclusive prefix sums
    __shared__ int32_t warp_part[32];
    __shared__ int32_t s_min, s_total;
    const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t* table = tables_cur_req0 + r * table_req_stride;
    int32_t* sidx = sidx_req0 + r * sidx_req_stride;
    int32_t* ulist = ulist_req0 + r * ulist_req_stride;
    int32_t* urep = urep_req0 + r * ulist_req_stride;
    int32_t* uoff = uoff_req0 + r * uoff_req_stride;
    const int ipt = (max_beam + 1023) / 1024;   // marks per thread in the scan
    int32_t off = 0;
    if (tid == 0) uoff[0] = 0;
    for (int level = 0; level < depth - 1; ++level) {
        const int32_t* row = table + (long long)level * max_beam;
        int32_t mn = 0x7fffffff;
        for (int b = tid; b < W; b += 1024) mn = min(mn, row[b]);
        for (int o = 16; o > 0; o >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        if (lane == 0) warp_part[warp] = mn;
        for (int i = tid; i < max_beam; i += 1024) marks[i] = 0;
        __syncthreads();
        if (warp == 0) {
            int32_t m = warp_part[lane];
            for (int o = 16; o > 0; o >>= 1) m = min(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == 0) s_min = m;
        }
        __syncthreads();
        mn = s_min;
        for (int b = tid; b < W; b += 1024) marks[row[b] - mn] = 1;
        __syncthreads();
        // exclusive scan of marks: thread t owns marks [t*ipt, (t+1)*ipt)
        int32_t local = 0;
        for (int j = 0; j < ipt; ++j) {
            const int i = tid * ipt + j;
            if (i < max_beam) local += marks[i];
        }
        int32_t incl = local;
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        __syncthreads();                       // warp_part is reused
        if (lane == 31) warp_part[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int32_t w = warp_part[lane], wi = w;
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t t = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += t;
            }
            warp_part[lane] = wi - w;          // exclusive prefix of the warp totals
            if (lane == 31) s_total = wi;
        }
        __syncthreads();
        int32_t pos = warp_part[warp] + incl - local;
        for (int j = 0; j < ipt; ++j) {
            const int i = tid * ipt + j;
            if (i < max_beam) {
                const int32_t m = marks[i];
                marks[i] = pos;                // now the rank of slot mn + i among the distinct slots
                if (m) ulist[off + pos] = mn + i;
                pos += m;
            }
        }
        __syncthreads();
        for (int b = tid; b < W; b += 1024) {
            const int32_t pos_b = off + marks[row[b] - mn];
            sidx[(long long)level * max_beam + b] = pos_b;
            urep[pos_b] = b;     // any of the beams that share the record will do: they share all its ancestors
        }
        off += s_total;
        if (tid == 0) uoff[level + 1] = off;
        __syncthreads();
    }
    // Compact copies for the shared-chains decode kernel (meaningful while the request has at most 255 distinct
    // records; the kernel checks the count): every beam's list position per level as one byte, rows padded with the
    // last live beam's; and per distinct record its level and its ancestors' list positions (through one of the
    // beams that hold it).
    uint8_t* sg8 = sg8_req0 + r * sg8_req_stride;
    for (int i = tid; i < (depth - 1) * sg_stride; i += 1024) {
        const int level = i / sg_stride, b = i - level * sg_stride;
        sg8[i] = (uint8_t)sidx[(long long)level * max_beam + min(b, W - 1)];
    }
    uint8_t* unode = unode_req0 + (long long)r * (ONELA_UNODE_CAP * 16);
    for (int j = tid; j < min(off, ONELA_UNODE_CAP); j += 1024) {
        int lv = 0;
        for (int l = 1; l < depth - 1; ++l) lv += (j >= uoff[l]) ? 1 : 0;
        const int rp = urep[j];
        uint32_t w[4] = {0u, 0u, (uint32_t)lv, 0u};
        for (int l = 0; l < min(lv, 8); ++l)
            w[l >> 2] |= ((uint32_t)sidx[(long long)l * max_beam + rp] & 0xffu) << (8 * (l & 3));
        reinterpret_cast<uint4*>(unode)[j] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace

cudaError_t launch_dedupe(const int32_t* tables_cur_req0, long long table_req_stride, int32_t* sidx_req0,
                          long long sidx_req_stride, int32_t* ulist_req0, long long ulist_req_stride,
                          int32_t* urep_req0, int32_t* uoff_req0, long long uoff_req_stride, uint8_t* sg8_req0,
                          long long sg8_req_stride, int32_t sg_stride, uint8_t* unode_req0, int32_t req_count, int32_t W,
                          int32_t depth, int32_t max_beam, cudaStream_t stream) {
    const size_t smem = sizeof(int32_t) * (size_t)max_beam;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(dedupe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dedupe_kernel<<<req_count, 1024, smem, stream>>>(tables_cur_req0, table_req_stride, sidx_req0, sidx_req_stride,
                                                     ulist_req0, ulist_req_stride, urep_req0, uoff_req0, uoff_req_stride, sg8_req0,
                                                     sg8_req_stride, sg_stride, unode_req0, W, depth, max_beam);
    return cudaGetLastError();
}

cudaError_t launch_reorder(int32_t* tables_req0, long long table_req_stride, int32_t req_count,
                           const int32_t* parents, int32_t W_new, int32_t W_prev, int32_t depth_old,
                           int32_t max_beam, int32_t max_steps, const BatchBases& bases, int32_t* status,
                           cudaStream_t stream) {
    dim3 grid((W_new + 255) / 256, depth_old + 1, req_count);
    reorder_kernel<<<grid, 256, 0, stream>>>(tables_req0, table_req_stride, parents, W_new, W_prev, depth_old,
                                             max_beam, max_steps, bases, status);
    return cudaGetLastError();
}

cudaError_t launch_export_chains(const int32_t* table_cur, int32_t W, int32_t depth, int32_t max_beam,
                                 int32_t* slots_out, cudaStream_t stream) {
    const int n = W * depth;
    export_chains_kernel<<<(n + 255) / 256, 256, 0, stream>>>(table_cur, W, depth, max_beam, slots_out);
    return cudaGetLastError();
}

}  // namespace onela
