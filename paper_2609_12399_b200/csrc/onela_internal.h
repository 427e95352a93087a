// Internal declarations shared by the host-side context (onela_api.cu) and the kernel files.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "onela.h"

namespace onela {

// Device addresses of the sub-buffers carved out of the caller's workspace.
struct Layout {
    int32_t* status;   // [4]: code, detail, spare, spare
    int32_t* tables;   // [request][2][max_steps][max_beam] global slot ids (double-buffered per request)
    int32_t* sidx;     // [request][max_steps][max_beam] per (level, beam): index into the request's distinct-record list
    int32_t* ulist;    // [request][max_steps*max_beam] distinct record slots of the live chains, oldest level first
    int32_t* uoff;     // [request][max_steps+1] start of each level inside ulist (uoff[level+1] = end)
    int32_t* urep;     // [request][max_steps*max_beam] per distinct record: one live beam whose chain holds it
    uint8_t* sg8;      // [request][max_steps][sg_stride] sidx as bytes, rows padded with the last live beam's entry
    uint8_t* unode;    // [request][ONELA_UNODE_CAP][16] per distinct record: ancestors' list positions (bytes 0-7), level (byte 8)
    float* s0;         // [request][layer][head][dv*dk] fp32
    float2* gates;     // [layer][head][arena_slots] (alpha, beta)
    char* kv;          // [layer][head][arena_slots][dk + dv] in rec_dtype: one row = k | v of one record
                       // (grouped value heads: keys only, [layer][key head][arena_slots][dk])
    char* vv;          // grouped value heads only: values [layer][value head][arena_slots][dv]
    unsigned long long* select_scratch;   // [request][ONELA_SELECT_PARTS][ONELA_SELECT_CAP]: partial results of beam selection
    float* s0_scale;   // [request][layer][head]: the power of two that brings the head's largest |S_0| element into
                       // [2^11, 2^12) (1 for an all-zero or non-finite state); written with the state, read by the
                       // tensor-core kernel, whose fp16 operand it keeps in range
    uint16_t* s0_f16;  // configurations of the tiled tensor-core kernel only: [request][layer][head] the state as that
                       // kernel's MMA operand - fp16, times the head's operand scale, value rows padded to a multiple
                       // of 128, in tiles of 128 rows x 64 columns (16 KB, rows of 128 bytes, 16-byte chunks swizzled
                       // by the row) in the order [tile of rows][tile of columns]; written with the state
    size_t total_bytes;
};
// bytes of one head's operand copy (see Layout::s0_f16)
inline size_t s0_f16_head_bytes(int32_t dk, int32_t dv) { return (size_t)((dv + 127) / 128) * 128 * (size_t)dk * 2; }

struct BatchBases {
    int32_t base[ONELA_MAX_BATCH];  // first slot of this call's records, per request of the batch
};

// Everything a decode kernel needs, passed by value as the kernel parameter.
struct DecodeArgs {
    const void* q;          // [req_count][W][H][dk]
    void* out;              // [req_count][W][H][dv]
    const void* k_in;       // fused append: this call's records [req_count][W][H][dk], [..][dv], gates [..][H];
    const void* v_in;       //   null for a plain decode (the newest record is then read from the arena)
    const float* alpha_in;
    const float* beta_in;
    char* kv_out;           // fused append: arena plane to write (same plane as kv)
    float2* gates_out;
    const float* s0;        // store slot of (req_begin, layer)
    const char* kv;         // arena plane of this layer
    const float2* gates;    // gate plane of this layer
    const int32_t* table;   // current ancestry buffer of req_begin: [level][max_beam]
    int32_t* status;
    long long s0_req_stride;     // floats between consecutive requests' store slots (same layer)
    long long table_req_stride;  // ints between consecutive requests' tables
    long long arena_slots;
    const int32_t* sidx;    // distinct-record index of req_begin (see Layout)
    const int32_t* ulist;
    const int32_t* uoff;
    const int32_t* urep;
    const uint8_t* sg8;     // byte copies of sidx and the per-record table (see Layout), of req_begin
    const uint8_t* unode;
    long long sg8_req_stride;
    int32_t sg_stride;
    long long sidx_req_stride, ulist_req_stride, uoff_req_stride;
    int32_t req_count, W, H, depth, max_beam;
    BatchBases bases;
    // grouped value heads (tensor-core kernel only; H above is then the number of VALUE heads): kv / kv_out are the
    // layer's key plane [Hk][arena_slots][dk], vv / vv_out its value plane [H][arena_slots][dv]; q and k_in have Hk heads
    const char* vv;
    char* vv_out;
    int32_t Hk, g;
    // ... and value widths of 256 / 512 (grouped or not): every value head is cut into `tiles` heads of 128 outputs, so
    // H = tiles * (value heads) and g = tiles * (value heads per key head); k_stride / v_stride: bytes between
    // consecutive slots of a key head's keys and of a value head's values (from kv and vv: one interleaved plane or two)
    int32_t tiles;
    long long k_stride, v_stride;
    // tensor-core kernel: per-head operand scale of S_0 (see Layout), entry of (req_begin, layer, head 0)
    const float* s0_scale;
    long long s0_scale_req_stride;
    // 1 when the launch that precedes this one on the context was a decode launch as well (of another layer or of
    // this one): nothing that launch wrote is read here except the caller's tensors, so a programmatic dependent
    // launch may read the index arrays, S_0 and the older records before it waits for its predecessor
    int32_t early_ok;
};

// Grouped value heads (Hv = g * Hk): what the grouped decode kernel needs.
struct GroupedArgs {
    const void* q;          // [req_count][W][Hk][dk]
    void* out;              // [req_count][W][Hv][dv]
    const float* s0;        // store slot of (req_begin, layer): [Hv][dv][dk]
    const char* kplane;     // this layer's keys   [Hk][arena_slots][dk]
    const char* vplane;     // this layer's values [Hv][arena_slots][dv]
    const float2* gates;    // this layer's gates  [Hv][arena_slots]
    const int32_t* table;   // current ancestry buffer of req_begin
    long long s0_req_stride, table_req_stride, arena_slots;
    int32_t req_count, W, Hk, g, depth, max_beam;
    BatchBases bases;
};
bool decode_grouped_supported(int32_t dk, int32_t dv);
cudaError_t launch_decode_grouped(const GroupedArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                                  cudaStream_t stream);
cudaError_t launch_append_grouped(const void* k, const void* v, const float* alpha, const float* beta, char* kplane,
                                  char* vplane, float2* gates, long long arena_slots, int32_t req_count, int32_t W,
                                  int32_t Hk, int32_t g, int32_t dk, int32_t dv, int32_t elem_bytes, const BatchBases& bases,
                                  cudaStream_t stream);

// Tiled tcgen05 decode kernel (onela_decode_tiled.cu): every supported shape from 64 x 64 up in either record dtype,
// grouped value heads or not.  Keys and values are addressed through planes and per-slot strides, so one struct serves
// the interleaved arena (kplane = the layer's k | v rows, vplane = kplane + dk elements, both strides dk + dv) and the
// split one (grouped value heads: two planes, strides dk and dv).
struct TiledArgs {
    const void* q;          // [req_count][W][Hk][dk]
    void* out;              // [req_count][W][Hv][dv]
    const void* k_in;       // fused append: this call's records [req_count][W][Hk][dk], [..][Hv][dv], gates [..][Hv], which
    const void* v_in;       //   the launch also writes to their arena slots; null for a plain decode (the newest record
    const float* alpha_in;  //   is then read from the arena)
    const float* beta_in;
    const float* s0;        // store slot of (req_begin, layer): [Hv][dv][dk]
    const float* s0_scale;  // operand scale of (req_begin, layer, value head 0) (see Layout)
    const char* s0_f16;     // operand copy of (req_begin, layer, value head 0) (see Layout::s0_f16)
    long long s0_f16_req_stride;   // bytes between consecutive requests' copies (same layer)
    char* kplane;           // key of (key head hk, slot) at kplane + ((hk * arena_slots + slot) * k_stride) elements
    char* vplane;           // value of (value head hv, slot) at vplane + ((hv * arena_slots + slot) * v_stride) elements
    float2* gates;          // [Hv][arena_slots]
    const int32_t* table;   // current ancestry buffer of req_begin
    int32_t* status;
    long long s0_req_stride, s0_scale_req_stride, table_req_stride, arena_slots, k_stride, v_stride;
    int32_t req_count, W, Hk, g, depth, max_beam;
    int32_t delta;          // 1: the arena keeps (alpha, delta, k) records and the launch replays both projections forward
    BatchBases bases;
};
bool decode_tiled_supported(int32_t dk, int32_t dv);
cudaError_t launch_decode_tiled(const TiledArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                                cudaStream_t stream);

// index kernels
cudaError_t launch_reorder(int32_t* tables_req0, long long table_req_stride, int32_t req_count,
                           const int32_t* parents, int32_t W_new, int32_t W_prev, int32_t depth_old,
                           int32_t max_beam, int32_t max_steps, const BatchBases& bases, int32_t* status,
                           cudaStream_t stream);
// Distinct-record index of the CURRENT ancestry table (levels 0 .. depth-2; the newest level is the
// beams' own records, all distinct): per level the sorted distinct slots and, per beam, where its
// ancestor sits in the request's concatenated list.  Integer work only.
// urep: per distinct record, one of the live beams whose chain holds it (all such beams share its older ancestors).
// sg8 / unode: byte-sized copies for the shared-chains kernel (see Layout).
#define ONELA_UNODE_CAP 256
inline int32_t sg_row_stride(int32_t max_beam) { return (max_beam + 64 + 15) & ~15; }
cudaError_t launch_dedupe(const int32_t* tables_cur_req0, long long table_req_stride, int32_t* sidx_req0,
                          long long sidx_req_stride, int32_t* ulist_req0, long long ulist_req_stride,
                          int32_t* urep_req0, int32_t* uoff_req0, long long uoff_req_stride, uint8_t* sg8_req0,
                          long long sg8_req_stride, int32_t sg_stride, uint8_t* unode_req0, int32_t req_count, int32_t W,
                          int32_t depth, int32_t max_beam, cudaStream_t stream);
cudaError_t launch_export_chains(const int32_t* table_cur, int32_t W, int32_t depth, int32_t max_beam,
                                 int32_t* slots_out, cudaStream_t stream);

// global beam selection: the W_new best (parent, code) pairs per request, best first (see onela_select.cu).
// `scratch` ([request][ONELA_SELECT_PARTS][ONELA_SELECT_CAP] 64-bit words) is used when a request has more than
// 4096 candidates; at most ONELA_SELECT_PARTS * 4096 candidates per request.
#define ONELA_SELECT_CAP 1024
#define ONELA_SELECT_PARTS 256
cudaError_t launch_select(const float* beam_scores, const float* cand_logp, int32_t req_count, int32_t W_prev, int32_t C,
                          int32_t W_new, unsigned long long* scratch, int32_t* parents, int32_t* codes, float* scores,
                          cudaStream_t stream);

// record / state kernels
cudaError_t launch_append(const void* k, const void* v, const float* alpha, const float* beta, char* kv_plane,
                          float2* gate_plane, long long arena_slots, int32_t req_count, int32_t W, int32_t H,
                          int32_t dk, int32_t dv, int32_t elem_bytes, const BatchBases& bases,
                          cudaStream_t stream);
// copies n_heads states of dv x dk floats and leaves each head's operand scale (see Layout::s0_scale) in scale_out
cudaError_t launch_store_state(const float* S0_in, float* slot, float* scale_out, long long n_heads, int32_t dk, int32_t dv,
                               cudaStream_t stream);
// the tiled kernel's operand copy of n_heads stored states (see Layout::s0_f16), from the store slots and their scales
cudaError_t launch_pack_state(const float* slot, const float* scale, uint16_t* dst, long long n_heads, int32_t dk, int32_t dv,
                              cudaStream_t stream);
cudaError_t launch_export_state(const float* slot, float* S0_out, int32_t H, int32_t dk, int32_t dv, cudaStream_t stream);
// returns cudaErrorInvalidValue with *supported = false when (dk, dv, dtype) has no instantiation
cudaError_t launch_prefill(const void* k, const void* v, const float* alpha, const float* beta, float* slot,
                           float* scale_out, int32_t n_tokens, int32_t H, int32_t dk, int32_t dv, int32_t rec_dtype,
                           bool* supported, cudaStream_t stream);

// decode kernels
cudaError_t launch_decode_generic(const DecodeArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype,
                                  int32_t out_dtype, bool* supported, cudaStream_t stream);
bool decode_generic_supported(int32_t dk, int32_t dv, int32_t rec_dtype);
// tcgen05 tensor-core kernel (sm_100a): dk = dv = 128, bf16 records
// forward projection replay over (alpha, delta, k) records (ONELA_FLAG_GTR_DELTA): append + decode of one layer
cudaError_t launch_decode_gtr(const DecodeArgs& a, int32_t dk, int32_t dv, int32_t rec_dtype, int32_t out_dtype,
                              bool* supported, cudaStream_t stream);
bool decode_sm100_supported(int32_t dk, int32_t dv, int32_t rec_dtype);
// delta_records: the arena keeps (alpha, delta, k) and the launch replays both projections forward (fused append only)
cudaError_t launch_decode_sm100_ws(const DecodeArgs& a, int32_t out_dtype, bool grouped, bool delta_records, cudaStream_t stream);

// Contiguous ranges of beam groups, one per CTA of a persistent decode kernel (host-side partitioner in
// onela_decode_sm100.cu): CTA c works on groups [begin[c], begin[c + 1]).
constexpr int DECODE_MAX_CTAS = 160;
struct DecodePartition {
    int32_t begin[DECODE_MAX_CTAS + 1];
};
// group_cost / seg_cost: relative cost of one group and of starting a (request, head) segment.  Returns the CTA count.
int make_decode_partition(int total_groups, int groups_per_pair, int sms, int group_cost, int seg_cost, DecodePartition* part);
int decode_sm_count();

// tcgen05 kernel for chains with heavily shared ancestors (dk = dv = 128, bf16 records, one key head per value head):
// the older levels of all chains are applied in compact form on the tensor cores (see onela_decode_wy.cu).
// Usable when every request of the call has at most WY_MAX_NODES distinct older records, at most WY_MAX_DEEP of them
// older than the beams' parents, and 2 <= depth <= WY_MAX_LEVELS + 1; the kernel checks the first two on the device.
constexpr int WY_MAX_NODES = 160, WY_MAX_DEEP = 64, WY_MAX_LEVELS = 8;
cudaError_t launch_decode_wy(const DecodeArgs& a, int32_t out_dtype, cudaStream_t stream);

}  // namespace onela
