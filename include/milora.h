/*
 * milora.h - C ABI of the MiLoRA adapter-apply library for NVIDIA B200 (sm_100a).
 *
 * The library implements the serving hot path of MiLoRA ("Mixture of Low-Rank
 * Adaptation", prompt-aware routing):
 *
 *   - Section 3.3, Eq. 2-3: once per prompt and per Transformer layer, pool the prompt's
 *     hidden states H^l, apply the activation g, multiply by the router weight W_r^l
 *     (d x 7), softmax, and select the top-scoring of the 7 LoRA positions
 *     q,k,v,o,gate,up,down.  The decision is stored in an int32 route table and reused
 *     for every generated token of that request.
 *   - Section 3.1, Eq. 1: x' = x W_m + s x W_m^A W_m^B + b_m is applied only on the selected
 *     module m of each request.  The caller computes x W_m + b_m; the library adds the
 *     LoRA term in place.
 *   - Section 4.5 (efficiency analysis): adapters are not merged into the backbone, so one
 *     batch mixes many tenants; tokens are bucketed by (module, tenant) first.
 *
 * Conventions
 *   - Plain C.  Every function returns a milora_status (MILORA_OK = 0) and never aborts,
 *     throws or exits.  Errors that the host can detect are reported before anything is
 *     launched.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *     The caller owns every buffer it passes; the library borrows it until the work
 *     enqueued by that call has finished on the stream.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All device
 *     work is enqueued on it and the call returns without waiting, except where stated.
 *   - Matrices are dense row-major.  Element type of activations, adapters and router
 *     weights is the context's dtype (fp32 or bf16); accumulation is always fp32.
 *   - A context is not thread-safe; use one per host thread or lock around it.
 *   - The compute calls of one context share scratch buffers that the library owns and grows on demand (router
 *     partial sums, prefill partial products, the fused projection's piece images, the decode kernels' counters
 *     and partial sums): order all compute calls of a context on ONE stream.  Two calls on different streams would
 *     race on the scratch, and a growth (cudaFree / cudaMalloc after synchronising the call's own stream) could
 *     free a buffer that a kernel on the other stream still reads.
 *   - Device-side index problems (a slot id out of range inside a device array) never
 *     fault: the offending item is skipped and a flag is raised that milora_poll_error reads.
 */
#ifndef MILORA_H_
#define MILORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct milora_ctx milora_ctx;

typedef enum {
  MILORA_OK = 0,
  MILORA_E_ARG = 1,          /* null pointer, negative size, index out of range            */
  MILORA_E_SHAPE = 2,        /* dimension not supported (see milora_create)                 */
  MILORA_E_DTYPE = 3,
  MILORA_E_UNREGISTERED = 4, /* tenant / adapter / router / slot not registered             */
  MILORA_E_CAPACITY = 5,     /* exceeds max_rank / max_tenants / max_requests / workspace   */
  MILORA_E_STATE = 6,
  MILORA_E_CUDA = 7,         /* a CUDA runtime call failed; see milora_last_cuda_error      */
  MILORA_E_DEVICE_INDEX = 8  /* reported by milora_poll_error: a kernel skipped a bad index */
} milora_status;

typedef enum { MILORA_F32 = 0, MILORA_BF16 = 1 } milora_dtype;

/* Section 3.3, Eq. 2: (b) average, (a) last-token, (c) max, (d) self-attention pooling (Appendix C). */
typedef enum { MILORA_POOL_MEAN = 0, MILORA_POOL_LAST = 1, MILORA_POOL_MAX = 2, MILORA_POOL_SELFATTN = 3 } milora_pool;

/* Activation g before the router (Section 3.3); RATIONAL is Eq. 7. */
typedef enum { MILORA_ACT_TANH = 0, MILORA_ACT_IDENTITY = 1, MILORA_ACT_RELU = 2, MILORA_ACT_GELU = 3,
               MILORA_ACT_RATIONAL = 4 } milora_act;

/* Section 3.1: module order 0..6; N_mod = 7. */
enum { MILORA_Q = 0, MILORA_K = 1, MILORA_V = 2, MILORA_O = 3, MILORA_GATE = 4, MILORA_UP = 5, MILORA_DOWN = 6,
       MILORA_NMOD = 7 };

enum { MILORA_MAX_RATIONAL_COEF = 16 };

/* How a selected module's LoRA term is weighted (Eq. 3 selects; the paper prints no weighting, so NONE is the
 * default reading).  PROB multiplies the term of the j-th selected module by its softmax probability. */
typedef enum { MILORA_GATE_NONE = 0, MILORA_GATE_PROB = 1 } milora_gate;

typedef struct {
  int n_layers;
  int d_model;      /* hidden size d; d_model, d_ff and d_kv must be multiples   */
  int d_ff;         /* of 8 (bf16) or 4 (fp32) so that rows are 16-byte aligned, */
  int d_kv;         /* else MILORA_E_SHAPE.  d_kv = output size of k and v.      */
  milora_dtype dtype;
  int max_rank;     /* largest LoRA rank that will be registered (1..256)       */
  int max_tenants;
  int max_requests; /* number of request slots (rows of the route table)        */
  int top_k;        /* k of Eq. 3 (Top-k): modules selected per request and layer, 1..7; 0 means 1 */
  int gate;         /* milora_gate                                               */
} milora_model_desc;

/* Create / destroy.  milora_create allocates the device tables (adapter table, router table,
 * slot table, route table [max_requests][n_layers][top_k] initialised to -1, gate table of the same
 * shape) with cudaMalloc on the current device and waits for their initialisation.  milora_destroy frees everything the
 * library allocated, including adapter copies. */
milora_status milora_create(const milora_model_desc* desc, milora_ctx** out);
milora_status milora_destroy(milora_ctx* ctx);
const char* milora_status_string(milora_status s);
/* Text of the last CUDA runtime error seen by this context ("" if none). */
const char* milora_last_cuda_error(const milora_ctx* ctx);

/* (d1, d2) of W_m for module m (Section 3.1): q,o d x d; k,v d x d_kv; gate,up d x d_ff; down d_ff x d. */
milora_status milora_module_dims(const milora_ctx* ctx, int module, int* d1, int* d2);

/* ---- adapter table (Eq. 1) ---------------------------------------------------------------
 * Register W^A (A_dev: d1 x rank) and W^B (B_dev: rank x d2), in the paper's orientation, for
 * (tenant, layer, module) with LoRA scale s (Eq. 1 is s = 1).  The library copies both into
 * its own pool in its own layout (A transposed to rank x d1) on `stream`; the caller may free
 * A_dev/B_dev once that stream work has finished.  Registering the same key again replaces it
 * (the caller must make sure no apply call using the old copy is still running). */
milora_status milora_register_adapter(milora_ctx* ctx, int tenant, int layer, int module, int rank, float scale,
                                      const void* A_dev, const void* B_dev, void* stream);

/* ---- router table (Eq. 2-3) --------------------------------------------------------------
 * Register the router of (tenant, layer): Wr_dev is d x 7 (paper orientation, context dtype);
 * bias_dev is 7 fp32 values or NULL (the paper prints no bias); Wsa_dev (d values, context
 * dtype) is required only for MILORA_POOL_SELFATTN; coef_host holds a_0..a_{n_a-1} then
 * b_1..b_{n_b} (host floats, n_a + n_b <= MILORA_MAX_RATIONAL_COEF) only for
 * MILORA_ACT_RATIONAL.  Everything is copied on `stream`. */
milora_status milora_register_router(milora_ctx* ctx, int tenant, int layer, const void* Wr_dev,
                                     const float* bias_dev, milora_pool pool, const void* Wsa_dev, milora_act act,
                                     const float* coef_host, int n_a, int n_b, void* stream);

/* Drop every adapter and router of a tenant (host-side table update; takes effect for calls
 * made afterwards).  Fails with MILORA_E_STATE while a request slot is bound to the tenant.  The tenant's copies
 * go back to the library's pool, from which later registrations are served first, so a server that admits and drops
 * tenants does not grow; the caller must make sure that no call that could still read them (an apply on a group
 * block built while the tenant was registered) is running or will be made. */
milora_status milora_unregister_tenant(milora_ctx* ctx, int tenant);
/* Bytes of the library's pool that registered adapters and routers occupy right now (copies in the library's
 * layouts: A^T and B row-major, plus, in bf16 contexts whose dimensions allow it, the two operand images: twice
 * the adapter's own size). */
milora_status milora_resident_bytes(const milora_ctx* ctx, size_t* adapter_pool_bytes);

/* ---- request slots -----------------------------------------------------------------------
 * Bind a slot to a tenant when a request is admitted; release it when the request ends.
 * Opening a slot resets its route row to -1 (not routed). */
milora_status milora_request_open(milora_ctx* ctx, int slot, int tenant);
milora_status milora_request_close(milora_ctx* ctx, int slot);

/* ---- routing (Section 3.3, Eq. 2-3; computed once per prompt, then reused) ----------------
 * Route P prompts at `layer`.  H_dev holds the prompts' hidden states back to back:
 * rows [cu_seqlens[p], cu_seqlens[p+1]) of a [T_total, d_model] matrix belong to prompt p;
 * T_total = cu_seqlens[P] must be passed by the host.  seq_slot_dev[p] is the request slot of
 * prompt p (P <= 4096).  Writes route[slot][layer][0..top_k) (module ids 0..6 in descending order of
 * their logits, ties to the lower index; Eq. 3, and the k sweep of Section 4.5), the matching softmax
 * probabilities to the gate table and, when not NULL, logits_out_dev [P][7] fp32 (g(h) W_r + bias) and probs_out_dev [P][7] fp32 (their
 * softmax).
 * Prompts whose slot is closed or whose tenant has no router at this layer get route -1.
 * Two launches (streaming partial reduction, then one CTA per prompt); deterministic (fixed reduction
 * order, no atomics on data).  The first call, and any call with more
 * rows than every earlier one, grows an internal scratch buffer (cudaMalloc after a stream sync). */
milora_status milora_route(milora_ctx* ctx, int layer, const void* H_dev, const int32_t* cu_seqlens_dev,
                           const int32_t* seq_slot_dev, int P, int T_total, float* logits_out_dev,
                           float* probs_out_dev, void* stream);

/* Routing for callers that must not allocate device memory (the paper has no counterpart; this is a
 * deployment variant of milora_route).  milora_route grows a scratch buffer with cudaMalloc when a batch
 * is larger than any before it.  That is not possible for a caller that runs inside a serving engine
 * whose memory pool already owns the whole device, inside a region where the allocator is frozen, or on
 * a latency path where the implicit device synchronisation of cudaMalloc/cudaFree is not acceptable.
 * This entry point takes the same arguments and gives the same results, but keeps its scratch (partial
 * column sums and one scheduling word) in a fixed array inside the library image:
 *   - the array is 16 MiB + 16 KiB and is held by every GPU that loads the library until the process
 *     exits;
 *   - a call needs (T_total / 64 + P) * (d_model + 2) floats of it; a call that needs
 *     more than 4 Mi floats, or has P > 4096, is rejected with MILORA_E_CAPACITY before any launch;
 *   - the first call on a device looks up the array's device address (cudaGetSymbolAddress); the
 *     context's device must be current (else MILORA_E_STATE), and this first call should be made
 *     before any stream capture begins;
 *   - all calls, from every context on that device, share the array: its scheduling word is cleared on
 *     `stream` at the start of each call, but two calls that overlap on the GPU (different streams)
 *     race on it, so keep calls of this entry point ordered on one stream;
 *   - it calls no cudaMalloc, cudaFree or other allocating routine.  Pending table updates made by
 *     register/open/close calls are still copied to the device first, as in milora_route. */
milora_status milora_route_static(milora_ctx* ctx, int layer, const void* H_dev, const int32_t* cu_seqlens_dev,
                                  const int32_t* seq_slot_dev, int P, int T_total, float* logits_out_dev,
                                  float* probs_out_dev, void* stream);

/* Device pointer to the route table, int32 [max_requests][n_layers][top_k], read-only for callers. */
milora_status milora_route_table(const milora_ctx* ctx, const int32_t** table_dev);

/* Copy route rows [slot_begin, slot_begin + n_slots) to / from host memory (n_slots * n_layers * top_k int32).
 * Both wait for `stream` first and return when the copy is done.  Writing lets a caller restore
 * decisions that were computed earlier (for example after moving a request to another replica);
 * values must be -1 or 0..6, and the modules of one (slot, layer) cell distinct. */
milora_status milora_route_table_read(milora_ctx* ctx, int slot_begin, int n_slots, int32_t* rows_host, void* stream);
milora_status milora_route_table_write(milora_ctx* ctx, int slot_begin, int n_slots, const int32_t* rows_host,
                                       void* stream);
/* The same for the gate table (fp32, same shape as the route table): entry j is the softmax probability of
 * the j-th selected module, written by milora_route.  Only read by the library when gate = MILORA_GATE_PROB. */
milora_status milora_gate_table_read(milora_ctx* ctx, int slot_begin, int n_slots, float* rows_host, void* stream);
milora_status milora_gate_table_write(milora_ctx* ctx, int slot_begin, int n_slots, const float* rows_host,
                                      void* stream);

/* ---- grouping (multi-tenant batches, Section 4.5) ------------------------------------------
 * A step's tokens are n_seq sequences laid out back to back (rows [cu_seqlens[i], cu_seqlens[i+1])
 * of every X / Y matrix; n_seq <= 4096); a decode request is a sequence of length 1 (cu_seqlens_dev
 * == NULL means every sequence has length 1).  For layers [layer_begin, layer_begin + n_layers) the tokens are
 * bucketed by key = route[slot][layer][j] * max_tenants + tenant(slot); with top_k > 1 a token belongs to
 * one bucket per selected module (n_seq * top_k <= 4096).  A sequence whose slot is closed or not routed, or
 * whose tenant has no adapter on any of its selected modules, is excluded (n_excluded counts its tokens);
 * n_active counts (token, module) pairs.
 *
 * Output: one int32 block per layer in ws_dev (block l at ws_dev + l * ws_stride), laid out as
 * milora_group_layout describes:
 *   header[16]     [0] n_seg  [1] n_excluded tokens  [2] n_active tokens  [3] n_tiles  [4] n_gather
 *   mod_offset[8]  segment-index range of each module
 *   seg_key[]      key of every non-empty bucket, ascending
 *   seg_offset[]   bucket boundaries in perm
 *   perm[]         active token rows ordered by (module, tenant, row)
 * followed by the work lists the apply kernels consume (dense tiles of consecutive rows for
 * long sequences; gathered rows for short ones).
 *
 * A block depends on the batch (which slots, which row ranges), on the routes of its slots and on the adapters of
 * their tenants, and on nothing else.  Routes are written once per request (Section 3.3), so the block of a decode
 * batch stays valid from step to step: build it when the batch changes (a request joins or leaves, a slot is
 * reopened, one of its tenants registers an adapter again or is dropped) and reuse it for every step in between.
 * The grouping launch costs about as much as the decode apply of one layer; calling it every step doubles the
 * cost of a decode step for nothing. */
typedef struct {
  size_t header, mod_offset, mod_tile_offset, mod_gather_offset;
  size_t seg_key, seg_offset, perm, tiles, gather_rows, gather;
  size_t seq_tile;           /* [n_seq][8]: first dense tile of (sequence, module m) at [m], -1 if none; [7] = bit mask
                                of the modules that have tiles for the sequence */
  size_t total;              /* int32 elements of one layer block (multiple of 4) */
  int max_tiles, max_gather;
} milora_group_layout_t;

milora_status milora_group_layout(const milora_ctx* ctx, int n_seq, int T, milora_group_layout_t* out);

milora_status milora_group(milora_ctx* ctx, int layer_begin, int n_layers, const int32_t* cu_seqlens_dev,
                           const int32_t* seq_slot_dev, int n_seq, int T, int32_t* ws_dev, size_t ws_stride,
                           void* stream);

/* One layer's group block, as written by milora_group with the same n_seq and T. */
typedef struct {
  const int32_t* ws_dev;
  int n_seq;
  int T;
} milora_groups;

/* ---- apply (Eq. 1 on the selected module) ------------------------------------------------
 * X_dev [T][d1] inputs of module `module`; Y_dev [T][d2] holds x W_m + b_m on entry and
 * x W_m + b_m + s (x W^A) W^B on exit for the rows whose request routes to `module` at `layer`;
 * all other rows are left untouched (bit-identical).  milora_apply_decode processes the rows of
 * short sequences (the gathered work list: decode tokens), milora_apply_prefill the rows of long
 * sequences (dense tiles: prompt tokens); a mixed batch calls both. */
milora_status milora_apply_decode(milora_ctx* ctx, int layer, int module, const void* X_dev, void* Y_dev,
                                  const milora_groups* groups, void* stream);
milora_status milora_apply_prefill(milora_ctx* ctx, int layer, int module, const void* X_dev, void* Y_dev,
                                   const milora_groups* groups, void* stream);

/* Which kernels milora_apply_decode uses in a bf16 context (all compute the same Eq. 1; results agree to
 * rounding of the fp32 sums, and each is deterministic from call to call):
 *   MILORA_DECODE_CLUSTER  one launch; a cluster of eight CTAs per job exchanges partial sums of x W^A through
 *                          distributed shared memory.  Shortest latency when the step has few jobs.
 *   MILORA_DECODE_SPLIT    two launches (x W^A, then the product with W^B added into y), both plain streams over
 *                          equally sized units handed out by a counter, with the contractions on mma.sync tiles;
 *                          the r values per row in between go through a scratch buffer of the context (the
 *                          second launch takes them as bf16 value + bf16 remainder, i.e. to 2^-17), which the first call (and any call with a larger
 *                          batch than every earlier one) grows with cudaMalloc after a stream sync.  Highest
 *                          bandwidth when the step's adapters exceed what one wave of clusters covers.
 *   MILORA_DECODE_AUTO     (default) STREAM for batches of 96 sequences or more where the context allows it (see
 *                          STREAM); otherwise SPLIT when the work list has room for more than two jobs per SM (on
 *                          a B200: every smaller batch that mixes prompts with decode rows), else CLUSTER.
 *   MILORA_DECODE_STREAM   one persistent launch (one CTA per SM) whose warps each stream pieces of the adapters'
 *                          operand images through their own ring of shared-memory buffers (cp.async.bulk) and
 *                          contract them on mma.sync tiles; x W^A goes from its producers to the consumers of W^B
 *                          inside the launch (scratch buffer of the context, grown like SPLIT's).  It is the kernel
 *                          behind milora_apply_decode_layers.  Needs a bf16 context with d_model, d_ff and d_kv
 *                          multiples of 128 and max_rank <= 64; other contexts fall back to CLUSTER.
 * Calls of one context that use SPLIT or STREAM must be ordered on one stream (they share a scratch buffer).
 * Returns MILORA_E_ARG for another value.  fp32 contexts always use the generic kernel.
 */
typedef enum { MILORA_DECODE_AUTO = 0, MILORA_DECODE_CLUSTER = 1, MILORA_DECODE_SPLIT = 2, MILORA_DECODE_STREAM = 3 }
    milora_decode_path;
milora_status milora_set_decode_path(milora_ctx* ctx, milora_decode_path path);
/* The kernel set (CLUSTER, SPLIT or STREAM) that milora_apply_decode would use, with the current setting, for a bf16
 * batch of n_seq sequences and T rows whose shapes fit both; host arithmetic only. */
milora_status milora_decode_path_for(const milora_ctx* ctx, int n_seq, int T, milora_decode_path* out);

/* ---- a whole decode step in one launch (Eq. 1 on every layer; Section 3.3: routes are reused) --------
 * Applies Eq. 1 to the short sequences (decode rows) of n_layers layers with ONE persistent kernel launch.
 * Entry i describes one layer: its group block (written by milora_group for that layer) and, per module m,
 * the inputs X_dev[m] [T][d1(m)] and the outputs Y_dev[m] [T][d2(m)], updated in place on the rows whose request
 * selects m at that layer; a NULL pair skips the module.  The layers are processed concurrently, so no buffer
 * that one entry writes may be read or written by another entry (every layer its own Y; X may be shared).
 * This is the call for an engine that has the inputs of several layers at hand (LoRA terms applied after the
 * backbone's projections were computed, speculative or pipelined layers, benchmark chains); a layer-by-layer
 * engine passes one entry per call.  `layers` is host memory and is read before the call returns.
 * Uses the MILORA_DECODE_STREAM kernel when the context allows it (see milora_set_decode_path), otherwise, or when
 * the CLUSTER or SPLIT set is forced, one milora_apply_decode_multi per layer.  More than 40 layers, or more
 * scratch than 512 MB, are split into several launches.  The first call, and calls with larger batches, allocate
 * (scratch, a pinned staging buffer for the layer records); the records are re-sent to the device only when they
 * differ from the previous call's, so a decode loop over fixed buffers uploads nothing.  Every wait inside the
 * kernel is bounded; a wait that runs out raises the device error flag (milora_poll_error). */
typedef struct {
  int layer;
  milora_groups groups;
  const void* X_dev[MILORA_NMOD];
  void* Y_dev[MILORA_NMOD];
} milora_decode_layer;
milora_status milora_apply_decode_layers(milora_ctx* ctx, const milora_decode_layer* layers, int n_layers, void* stream);
/* Stages (16 KB pieces of an operand image) per work unit of the STREAM kernel: 1..64, or 0 (default) to let the
 * library choose from the batch size (long units for large batches, single stages for small ones). */
milora_status milora_set_decode_unit_stages(milora_ctx* ctx, int unit_stages);

/* Several module call sites of one layer in a single launch (for example q,k,v share an input,
 * gate,up share an input).  modules[i], X_dev[i], Y_dev[i] describe site i; a module may appear once. */
milora_status milora_apply_decode_multi(milora_ctx* ctx, int layer, int n_sites, const int* modules,
                                        const void* const* X_dev, void* const* Y_dev, const milora_groups* groups,
                                        void* stream);
milora_status milora_apply_prefill_multi(milora_ctx* ctx, int layer, int n_sites, const int* modules,
                                         const void* const* X_dev, void* const* Y_dev, const milora_groups* groups,
                                         void* stream);

/* Modules of one layer that read the SAME input matrix X_dev [T][d1] (q, k, v read the attention input; gate and up
 * the MLP input; all listed modules must have the same d1, else MILORA_E_ARG): Y_dev[i] [T][d2(modules[i])] +=
 * s (x W^A) W^B of module modules[i] on the rows whose request selects it (Eq. 1 with the routing of Section 3.3).
 * With top_k == 1 a row selects one module and this is milora_apply_prefill_multi.  With top_k > 1 a sequence
 * that selects several of the listed modules has every 128-row tile of X read once for all of them (up to three
 * modules per pass), instead of once per module.  milora_apply_prefill_multi does the same whenever it is given
 * equal X_dev pointers.  Results are those of separate milora_apply_prefill calls, bit for bit. */
milora_status milora_apply_prefill_shared(milora_ctx* ctx, int layer, int n_sites, const int* modules, const void* X_dev,
                                          void* const* Y_dev, const milora_groups* groups, void* stream);

/* ---- fused projection (Eq. 1 in one pass) ---------------------------------------------------------
 * Y_dev [T][d2] = X_dev [T][d1] . W_m + b_m for EVERY row of the step, plus s (x W^A) W^B on the rows of long
 * sequences (the dense tiles of `groups`) whose request selects `module` at `layer`: the backbone's own
 * projection and the LoRA term in one tensor-core kernel, so that Y is written once and never re-read.
 * Wt_dev is W_m transposed, [d2][d1] row-major (the layout in which an nn.Linear keeps its weight);
 * bias_dev is d2 values or NULL; all in bf16.  Rows of short sequences (the gathered list: decode tokens)
 * receive only the base projection here; follow with milora_apply_decode for their LoRA term.
 * When to use it: measured on a B200 at the LLaMA-2-7B sizes (32,768 rows), this call takes 0.09-0.11 ms (q site) to
 * 0.21 ms (down site) longer than a library GEMM of the base projection alone, while the separate
 * milora_apply_prefill for all seven call sites of the layer costs 0.22 ms in total; a caller whose own GEMM is as
 * fast as the library's should therefore keep it and call milora_apply_prefill afterwards.  The fused call pays
 * where the caller has no GEMM of that quality, or where Y must not be written twice.
 * Three launches (shrink, piece packing, persistent GEMM).  Returns MILORA_E_SHAPE unless the context is
 * bf16, max_rank <= 32, d1 is a multiple of 64, d2 a multiple of 256 and T >= 128; such callers use their own
 * GEMM followed by milora_apply_prefill.  Grows an internal scratch buffer like milora_route does. */
milora_status milora_linear_prefill(milora_ctx* ctx, int layer, int module, const void* X_dev, const void* Wt_dev,
                                    const void* bias_dev, void* Y_dev, const milora_groups* groups, void* stream);

/* ---- one step from host buffers ------------------------------------------------------------------
 * The whole path for one layer with every input in HOST memory (pinned memory makes the copies
 * asynchronous): copy in, route the prompts (Eq. 2-3), group the step's sequences, apply Eq. 1 on
 * every listed module for prompt rows and decode rows, copy the outputs back.  Everything is enqueued
 * on `stream`; the host buffers may be reused once the stream has been synchronised.
 *   n_prompts prompts to route: rows [cu_prompts_host[p], cu_prompts_host[p+1]) of H_host
 *             ([cu_prompts_host[n_prompts]][d_model]), slots prompt_slot_host[p]; n_prompts = 0 skips routing;
 *   n_seq sequences of T rows in total (cu_seq_host[n_seq+1], seq_slot_host[n_seq]) form the step;
 *   X_host[m] / Y_host[m] are the [T][d1(m)] inputs and [T][d2(m)] outputs of module m; a NULL pair skips m.
 * Only the rows the method touches cross the link.  After routing, the call reads the route table back to the
 * host (the one point where it waits for `stream`), and then, module by module, sends the X and Y rows of the
 * sequences that select that module (one copy per run of adjacent sequences), applies Eq. 1 and fetches the same
 * rows of Y.  Rows of sequences that do not select a module are never sent, and their rows of Y_host[m] keep what
 * they held.  The copy of one module's output back to the host runs on a stream of the library's own while the
 * next module is uploaded (the link carries both directions at once), and `stream` waits for the last of those
 * copies before the call's work counts as done on it.  The first call creates that stream and its events.
 * workspace_dev is caller-owned device memory of at least milora_step_host_workspace() bytes,
 * 256-byte aligned; the library allocates no device memory here except what milora_route may grow. */
typedef struct {
  int layer;
  int n_prompts;
  const int32_t* cu_prompts_host;
  const int32_t* prompt_slot_host;
  const void* H_host;
  int n_seq;
  int T;
  const int32_t* cu_seq_host;
  const int32_t* seq_slot_host;
  const void* X_host[MILORA_NMOD];
  void* Y_host[MILORA_NMOD];
} milora_host_step;

milora_status milora_step_host_workspace(const milora_ctx* ctx, const milora_host_step* step, size_t* bytes);
milora_status milora_step_host(milora_ctx* ctx, const milora_host_step* step, void* workspace_dev,
                               size_t workspace_bytes, void* stream);

/* Waits for `stream`, then reads and clears the device error flag.  *device_flag_out is 0 when no
 * kernel skipped anything; the return value is MILORA_E_DEVICE_INDEX otherwise. */
milora_status milora_poll_error(milora_ctx* ctx, int* device_flag_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MILORA_H_ */
