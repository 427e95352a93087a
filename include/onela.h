/*
 * onela.h - C ABI of the beam-shared Gated DeltaNet (GDN) decode library for NVIDIA B200 (sm_100a).
 *
 * The library holds, for every request, ONE post-prefill recurrent state S_0 per (layer, head)
 * (the shared context state is kept once, not per beam: paper Section 3.2), an append-only arena of per-token transition
 * records, and an ancestry index that maps every live beam to the records on its lineage
 * (Section 3.3, Eq. 5).  A decode call evaluates the GDN output of Eq. 1,
 *
 *        S_t = alpha_t S_{t-1} + beta_t (v_t - alpha_t S_{t-1} k_t) k_t^T ,    o_t = S_t q_t ,
 *
 * for every (beam, head) WITHOUT materialising any per-beam state: with
 * A_j = alpha_j (I - beta_j k_j k_j^T), Eq. 1 reads S_j = S_{j-1} A_j + beta_j v_j k_j^T, hence for any r
 * S_j r = S_{j-1} (A_j r) + beta_j (k_j . r) v_j.  Folding the query through the beam's records from
 * the newest to the oldest,
 *        r <- q ;   for j = t ... 0:   c = k_j . r ;  corr += beta_j c v_j ;  r <- alpha_j (r - beta_j c k_j) ,
 * gives o = S_0 r + corr, so all beams of a request meet S_0 in one dense [dv x dk] . [dk x W]
 * contraction per head.  (This is the adjoint of the paper's forward projection replay, Eq. 3-4;
 * the record kept here is the raw token (k, v, alpha, beta) rather than (alpha, delta, k).)
 *
 * Conventions
 *  - Every pointer whose name ends in _dev is DEVICE memory owned by the caller; *_host is host memory.
 *    The library allocates no device memory: the caller passes one workspace of
 *    onela_workspace_bytes() bytes (1024-byte aligned) at onela_create(); the library carves it into the
 *    S_0 store, the record arena, the ancestry tables and a status word.  The context itself is a small
 *    host object released by onela_destroy(), which never touches the workspace.
 *  - `stream` is a cudaStream_t passed as void*.  Every call is asynchronous and ordered on that
 *    stream; inputs may be reused as soon as the stream has passed the call.  Only
 *    onela_poll_device_status() synchronises.  The warp-specialised tensor-core decode kernel is launched with programmatic
 *    stream serialisation: it may start while the previous kernel of the stream drains, but it reads only its
 *    own shared-state store before it has waited for that kernel's completion, so stream order holds for every
 *    tensor the caller passes.  A caller kernel that follows it AND is itself launched with programmatic stream
 *    serialisation must wait for its grid dependency before it reads the decode outputs, as that launch mode
 *    requires of any kernel.
 *  - Tensors are dense, row-major, last index contiguous.  q, k, v use cfg.rec_dtype, outputs
 *    cfg.out_dtype, gates and S_0 are fp32.  All tensor pointers must be 16-byte aligned.
 *  - Errors the host can see return a negative status and launch nothing.  Errors only the device can
 *    see (a parent index outside the previous beam) set a sticky status word, the offending index is
 *    clamped to 0, and nothing traps.
 *  - Call order per request:  init/prefill_shared_state for each layer used (restarts the request at
 *    depth 0)  ->  repeat {  reorder_beams (once per decode call; shared by all layers and heads)  ->
 *    per layer { append_records exactly once  ->  decode_step any number of times } }, where
 *    append_decode_step stands for the layer's append and its first decode in one launch.  select_beams
 *    may run before a reorder_beams to produce its parents; release_request ends a request.
 *    Violations return ONELA_E_ORDER.
 *  - Slot numbering: one bump cursor per context.  reorder_beams over requests [b, b+n) assigns, in
 *    request order, base(req, t) = cursor, cursor += W_new (after a release_request: the lowest released
 *    range that fits, first).  The record of beam i at decode call t lives
 *    at global slot base(req, t) + i in every layer (a record is written once, at its decode call's slots, and
 *    never moves afterwards: Section 3.3).
 *  - Batched calls (req_count > 1) need the same beam width and depth on every request of the batch,
 *    and at most ONELA_MAX_BATCH requests.
 */
#ifndef ONELA_H
#define ONELA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct onela_ctx onela_ctx;
typedef int32_t onela_status;

#define ONELA_OK 0
#define ONELA_E_INVAL (-1)        /* null / shape / dtype / alignment / range */
#define ONELA_E_CAPACITY (-2)     /* arena, max_steps or max_beam exhausted */
#define ONELA_E_ORDER (-3)        /* call sequence violated */
#define ONELA_E_CUDA (-4)         /* a CUDA runtime call or launch failed */
#define ONELA_E_UNSUPPORTED (-5)  /* (dk, dv, dtype) combination not compiled */
#define ONELA_E_DEVICE_CHECK (-6) /* the device found a bad parent index (sticky) */
#define ONELA_E_TIMEOUT (-7)      /* a bounded device-side wait expired (sticky) */

#define ONELA_DTYPE_F32 0
#define ONELA_DTYPE_BF16 1

#define ONELA_MAX_BATCH 64

/* flags */
#define ONELA_FLAG_DRY_RUN 1u       /* validate and advance host bookkeeping, launch nothing (host-logic tests) */
#define ONELA_FLAG_FORCE_GENERIC 2u /* use the CUDA-core decode kernel (fp32 throughout) even where a tensor-core kernel applies */
/* Record format and replay order of Section 3.2 (Eq. 2-4): the arena keeps (alpha_t, delta_t, k_t) with
 * delta_t = beta_t (v_t - alpha_t S_{t-1} k_t) in rec_dtype in place of v_t, and a decode call replays the two
 * projection accumulators S q_t and S k_t forward from S_0 through the beam's records (oldest first).  delta_t
 * depends on the parent state, so records can only be produced where the replay runs: in this mode
 * onela_append_decode_step is the one call per layer and decode call; onela_append_records and onela_decode_step
 * return ONELA_E_UNSUPPORTED.  dk == dv in {32, 64, 128}; from 64 x 64 up both projections S q_t and S k_t of a beam go
 * through S_0 in one MMA set on the tensor cores (128 x 128 bf16 on the warp-specialised kernel, the rest on the tiled
 * one), 32 x 32 runs on CUDA cores.  Later calls replay the ROUNDED
 * delta, so with bf16 records the result drifts from the exact recurrence by about one bf16 rounding per record
 * (the default raw-record format has no such term). */
#define ONELA_FLAG_GTR_DELTA 4u
/* Chains that share most of their older records (few distinct ancestors per request: at most 160 distinct older
 * records, at most 64 of them older than the beams' parents, chains of at most 9 records): onela_decode_step and
 * onela_append_decode_step apply every level but the newest on the tensor cores (dk = dv = 128, bf16 records, one
 * key head per value head).  A call whose ancestry does not fit reports ONELA_E_UNSUPPORTED through the sticky
 * device status word and leaves its outputs unwritten. */
#define ONELA_FLAG_SHARED_CHAINS 8u

typedef struct onela_config {
    int32_t num_requests; /* request slots */
    int32_t num_layers;   /* GDN layers sharing the ancestry index */
    int32_t num_heads;    /* key heads (and value heads, unless num_v_heads says otherwise) */
    int32_t dk, dv;       /* head dimensions of k/q and of v/o: (32, 32), (64, 64), (128, 128), (128, 256), (256, 256),
                           * (128, 512) or (256, 512), else ONELA_E_UNSUPPORTED; dk = 128 with bf16 records runs on
                           * the warp-specialised tensor-core kernel at every value width (dv = 256 / 512 as two / four
                           * tiles of 128 outputs that share the key head's fold); every other shape from (64, 64) up,
                           * in either record dtype, on a tiled kernel whose contraction with S_0 runs on the tensor
                           * cores as well (fp16 operands kept in range by exact powers of two, fp32 accumulation);
                           * (32, 32) on CUDA cores in fp32 throughout */
    int32_t max_beam;     /* largest beam width W_t */
    int32_t max_steps;    /* largest number of decode calls per request (chain depth) */
    int32_t rec_dtype;    /* dtype of q, k, v: ONELA_DTYPE_* */
    int32_t out_dtype;    /* dtype of o */
    int64_t arena_slots;  /* record slots per layer, shared by all requests (< 2^31) */
    uint32_t flags;
    /* Grouped value heads (shapes of the operator suite of Section 4.1): 0 or num_heads = one value head per key
     * head; otherwise a multiple g * num_heads: value head j reads the queries and keys of key head j / g, while
     * states, values, gates and outputs are per value head.  Then q, k are [..][num_heads][dk]; v, alpha, beta, out
     * and S_0 are [..][num_v_heads][..]; a record keeps k once per key head and (v, alpha, beta) per value head
     * (num_heads * dk + num_v_heads * (dv + 8 bytes of gates) per slot instead of num_v_heads * (dk + dv + ..)).
     * (dk, dv) in {(64, 64), (128, 128), (128, 256)}: dk = 128 with bf16 records on the warp-specialised tensor-core
     * kernel, the rest on the tiled one; onela_prefill_shared_state and ONELA_FLAG_GTR_DELTA are not available
     * (ONELA_E_UNSUPPORTED). */
    int32_t num_v_heads;
} onela_config;

/* Bytes of device workspace the configuration needs; 0 if the configuration is invalid. */
size_t onela_workspace_bytes(const onela_config* cfg);

/* Build a context over a caller-owned workspace (device pointer, 1024-byte aligned, at least
 * onela_workspace_bytes(cfg) bytes).  Pure host work: nothing is launched; the first call that takes
 * a stream clears the status word on that stream.  The workspace must outlive the context. */
onela_status onela_create(const onela_config* cfg, void* workspace_dev, size_t workspace_bytes, onela_ctx** out);
onela_status onela_destroy(onela_ctx* ctx);

/* Forget every request and rewind the arena cursor to 0 (records are never reclaimed one by one:
 * the arena is append-only, Section 3.3). */
onela_status onela_reset(onela_ctx* ctx, void* stream);

/* Shared-state store (Section 3.2: the post-prefill state S_ctx is stored once per request).
 * Copies S0_dev [num_heads][dv][dk] fp32 into the store slot of (request, layer); the caller may free
 * S0_dev once the stream has passed the call.  Restarts the request at depth 0 if it had decoded. */
onela_status onela_init_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, const float* S0_dev,
                                     void* stream);

/* The same for ALL layers of req_count consecutive requests in one copy (a serving loop that admits a batch
 * stores num_layers states per request: one call instead of req_count * num_layers).  S0_dev (device, 16-byte
 * aligned) is [req_count][num_layers][value heads][dv][dk] fp32; same ownership and restart rule, applied to every
 * request of the range.  ONELA_E_INVAL for a range outside the request slots or a null / misaligned pointer, and
 * nothing is copied. */
onela_status onela_init_shared_states(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const float* S0_dev,
                                      void* stream);

/* Same store slot, filled by running Eq. 1 from the zero state over n_tokens prompt tokens in fp32:
 * k_dev [n_tokens][H][dk], v_dev [n_tokens][H][dv] in rec_dtype, alpha_dev, beta_dev [n_tokens][H] fp32. */
onela_status onela_prefill_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, const void* k_dev,
                                        const void* v_dev, const float* alpha_dev, const float* beta_dev,
                                        int32_t n_tokens, void* stream);

/* Read the store slot of (request, layer) back as S0_out_dev [num_heads][dv][dk] fp32 row-major, bit for
 * bit what was stored (the tensor-core kernel converts S_0 to scaled fp16 only on its way into tensor memory). */
onela_status onela_export_shared_state(onela_ctx* ctx, int32_t request, int32_t layer, float* S0_out_dev,
                                       void* stream);

/* Ancestry index update, Eq. 5 (Section 3.3): open decode call t for requests
 * [req_begin, req_begin+req_count) with W_new beams each.  parents_dev [req_count][W_new] int32 gives
 * pi_t(b), the parent of beam b in the previous beam; it must be NULL exactly when the requests are
 * at depth 0 (every beam's parent is S_0).  Writes indices only: new row b = parent's row, plus the
 * slot base(req, t) + b of the record about to be appended.  No record is moved or copied. */
onela_status onela_reorder_beams(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const int32_t* parents_dev,
                                 int32_t W_new, void* stream);

/* Give a finished request's record slots back (the paper is silent on reclamation; the reading taken: once a
 * request's generation is over its records are dead).  Host bookkeeping only: every slot range the request was
 * given by its reorder_beams calls returns to the context, the request drops its beams and its stored states (it
 * needs init/prefill_shared_state again before it decodes).  Later reorder_beams calls place a request's W_new
 * slots in the lowest released range that holds them and fall back on the bump cursor; ranges that touch are
 * merged, and a range that reaches the cursor lowers it.  Kernels already enqueued that read the released records
 * finish before later calls overwrite the slots as long as all calls go to one stream (or are ordered by events).
 * A request slot that is re-initialised WITHOUT being released keeps its old slots occupied until onela_reset. */
onela_status onela_release_request(onela_ctx* ctx, int32_t request);

/* Global beam selection feeding onela_reorder_beams (every live beam is extended by every code of the codebook and
 * the best k of all the candidates survive: Section 2.1): for each request of [req_begin, req_begin+req_count),
 * candidate (p, c) scores beam_scores_dev[req][p] + cand_logp_dev[req][p][c], added in fp32, with p over the
 * W_prev beams of the request's current decode call (W_prev = 1, the root, before the first call) and c over the C
 * codes.  The W_new best are written best first: parents_out_dev [req_count][W_new] int32 (the parent map pi_t in
 * the form reorder_beams takes), codes_out_dev [req_count][W_new] int32, scores_out_dev [req_count][W_new] fp32.
 * Equal scores go to the smaller flat index p * C + c; NaN ranks below every number; -0 equals +0.  Reads and
 * writes only the caller's buffers and changes no state of the context, so selection, reorder and the layers'
 * decode launches of a step can be captured in one CUDA graph.  1 <= W_new <= min(1024, W_prev * C), else
 * ONELA_E_CAPACITY. */
onela_status onela_select_beams(onela_ctx* ctx, int32_t req_begin, int32_t req_count, const float* beam_scores_dev,
                                const float* cand_logp_dev, int32_t C, int32_t W_new, int32_t* parents_out_dev,
                                int32_t* codes_out_dev, float* scores_out_dev, void* stream);

/* onela_select_beams for callers that cannot hand the library a workspace.  (The paper has no counterpart: this
 * is a packaging variant, not part of the method.)  Some hosts may not allocate device memory where selection
 * runs: a serving process that gave every byte of the GPU to its own pool at start-up, a plug-in that is called
 * on a stream it does not own and must not trigger cudaMalloc's device-wide synchronisation, a real-time loop
 * with an allocation ban.  They have no onela context either, so the call takes the shapes directly
 * (beam_scores_dev [req_count][W_prev], cand_logp_dev [req_count][W_prev][C], outputs [req_count][W_new], as in
 * onela_select_beams) and keeps its partial results in an array built into the library: 4 MiB of every GPU that
 * loads the library, held until the process exits.  Limits, fixed at build time: req_count <= 2,
 * W_prev * C <= 1,048,576 candidates per request, W_new <= 1024; anything larger returns ONELA_E_CAPACITY and
 * launches nothing (split the batch, or use onela_select_beams).  The call allocates nothing and frees nothing.
 * The first call on a device looks the array's device address up; make that call before any stream capture
 * begins on that device.  All calls share the one array: it keeps whatever the last call left (nothing in it has
 * to start at zero), and two calls that overlap on the GPU - different streams, or a call inside a graph that is
 * replayed while another call runs - race on it; keep them ordered on one stream or by events.  Results are those
 * of onela_select_beams, bit for bit. */
onela_status onela_select_beams_static(const float* beam_scores_dev, const float* cand_logp_dev, int32_t req_count,
                                       int32_t W_prev, int32_t C, int32_t W_new, int32_t* parents_out_dev,
                                       int32_t* codes_out_dev, float* scores_out_dev, void* stream);

/* Append this call's transition records for one layer (a call adds one compact record per beam and head; no full
 * recurrent state is ever written back: Section 3.4): k_dev [req_count][W][H][dk],
 * v_dev [req_count][W][H][dv] in rec_dtype, alpha_dev, beta_dev [req_count][W][H] fp32.  Values are
 * stored bit-exactly and never modified afterwards. */
onela_status onela_append_records(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                                  const void* k_dev, const void* v_dev, const float* alpha_dev,
                                  const float* beta_dev, void* stream);

/* Fused decode (Eq. 1 output through the backward fold described at the top): q_dev
 * [req_count][W][H][dk] in rec_dtype -> out_dev [req_count][W][H][dv] in out_dtype.  The chain of a beam
 * includes the record appended in this call (o_t reads the UPDATED state, Eq. 1). */
onela_status onela_decode_step(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                               const void* q_dev, void* out_dev, void* stream);

/* append_records and decode_step of one layer in ONE launch (the paper's kernel also appends the new
 * record inside the decode kernel, Section 3.4): the call's records are read from the caller's tensors,
 * folded as each beam's newest record, and written to the arena by the same kernel, so they cross HBM
 * once instead of three times.  Same arguments, checks and call-order rules as the two calls it replaces
 * (it counts as the layer's one append of this decode call; decode_step may still be called afterwards).
 * One launch on both tensor-core kernels; where a CUDA-core kernel runs (dk = dv = 32, ONELA_FLAG_FORCE_GENERIC)
 * the call is the copy kernel followed by the decode kernel. */
onela_status onela_append_decode_step(onela_ctx* ctx, int32_t req_begin, int32_t req_count, int32_t layer,
                                      const void* k_dev, const void* v_dev, const float* alpha_dev,
                                      const float* beta_dev, const void* q_dev, void* out_dev, void* stream);

/* Copy the ancestry rows of one request to slots_dev [W][depth] int32 (global slot ids, oldest first;
 * the last column is the beam's own record).  depth_host / width_host (host pointers, may be NULL)
 * receive the shape immediately. */
onela_status onela_export_chains(onela_ctx* ctx, int32_t request, int32_t* slots_dev, int32_t* depth_host,
                                 int32_t* width_host, void* stream);

/* Synchronise the device and read the sticky status word: *code_host is ONELA_OK,
 * ONELA_E_DEVICE_CHECK or ONELA_E_TIMEOUT; *detail_host the offending value.  Clears the word. */
onela_status onela_poll_device_status(onela_ctx* ctx, int32_t* code_host, int32_t* detail_host);

/* Resident bytes (host bookkeeping; Section 4.4 reports the same three quantities): the stored S_0
 * matrices (fp32; configurations of the tiled tensor-core kernel keep every state a second time as that kernel's
 * fp16 operand, half as many bytes again, not counted here), the records appended so far (slots * heads * record
 * bytes * layers), and the live ancestry rows. */
onela_status onela_get_stats(const onela_ctx* ctx, int64_t* s0_bytes_host, int64_t* arena_bytes_used_host,
                             int64_t* index_bytes_host);

/* First global slot of the records request `request` appended at decode call `step` (host bookkeeping). */
onela_status onela_get_step_base(const onela_ctx* ctx, int32_t request, int32_t step, int32_t* base_host);

/* Kernels this context has launched since creation (host counter; for launch accounting). */
int64_t onela_launch_count(const onela_ctx* ctx);

/* Which kernel decode_step of this context runs: 1 the warp-specialised tcgen05 kernel (dk = 128, bf16 records),
 * 2 the tiled tcgen05 kernel (every other shape from 64 x 64 up, either record dtype, grouped value heads or not),
 * 0 a CUDA-core kernel (dk = dv = 32, ONELA_FLAG_FORCE_GENERIC). */
int32_t onela_uses_tensor_core_path(const onela_ctx* ctx);

const char* onela_status_string(onela_status s);

#ifdef __cplusplus
}
#endif
#endif /* ONELA_H */
