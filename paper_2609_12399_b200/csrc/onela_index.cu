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

}  // namespace

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
