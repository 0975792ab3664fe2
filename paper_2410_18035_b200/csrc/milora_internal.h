// Internal declarations shared by the host code and the kernels of libmilora.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "milora.h"

namespace milora {

// ---- device-visible tables -------------------------------------------------------------
// One LoRA pair in library layout.  At is rank x d1 (W^A transposed), B is rank x d2, both row-major
// in the context dtype and 256-byte aligned.  At_img / B_img are the same matrices cut into the
// shared-memory operand images the tensor-core kernels fetch with one bulk copy per chunk (bf16
// contexts whose dimensions allow it; nullptr otherwise).
struct AdapterEntry {
  const void* At;
  const void* B;
  const void* At_img;
  const void* B_img;
  int32_t rank;      // 0 = not registered
  float scale;
  int32_t rank_pad;  // rank rounded up to a multiple of 16 (rows of the operand images)
  int32_t pad[5];
};
static_assert(sizeof(AdapterEntry) == 64, "AdapterEntry must stay 64 bytes");

// Router of one (tenant, layer): W is 7 x d (W_r transposed), context dtype.
struct RouterEntry {
  const void* W;      // nullptr = not registered
  const void* Wsa;    // d values, only for the self-attention pooler
  float bias[8];      // 7 used; zeros when the router has no bias
  float coef[MILORA_MAX_RATIONAL_COEF];
  int32_t pool, act, n_a, n_b;
};

constexpr int kHeaderInts = 16;
constexpr int kTileRows = 128;     // rows per dense tile (prefill path)
constexpr int kGatherRows = 4;     // rows per gather job (decode path)
constexpr int kLongSeq = 32;       // sequences of at least this many tokens go to dense tiles
constexpr int kMaxSeq = 4096;      // sequences per grouping / routing call
constexpr int kJobInts = 16;       // every job record is 64 bytes
enum HeaderSlot { H_NSEG = 0, H_NEXCL = 1, H_NACTIVE = 2, H_NTILES = 3, H_NGATHER = 4 };

// Work records written by the grouping kernel.  They carry the adapter pointers, so an apply kernel
// needs one 64-byte load to know its whole job.  They stay valid until an adapter of the batch is
// registered again or a slot of the batch is closed.
struct GatherJob {       // up to kGatherRows rows anywhere in X / Y that share an adapter
  const void* At;
  const void* B;
  int32_t rank;
  float scale;
  int32_t module, count;
  int32_t rows[kGatherRows];
  float gate[kGatherRows];   // per-row weight of the LoRA term (1 unless probability gating is on)
};
struct TileJob {         // `count` consecutive rows starting at `start`
  const void* At;
  const void* B;
  const void* At_img;
  const void* B_img;
  int32_t rank;
  float scale;
  int32_t module, count, seg, start, rank_pad;
  int32_t ent;             // bits 0..15: entry index (sequence * top_k + j); bits 16..22: modules with tiles for the sequence
};
static_assert(sizeof(GatherJob) == 64 && sizeof(TileJob) == 64, "job records are 64 bytes");

// Device error flag bits.
enum ErrBit { ERR_BAD_SLOT = 1, ERR_BAD_ROW = 2, ERR_WAIT_TIMEOUT = 4, ERR_BAD_ITEM = 8 };

struct DeviceTables {
  const AdapterEntry* adapters;   // [max_tenants][n_layers][7]
  const RouterEntry* routers;     // [max_tenants][n_layers]
  const int32_t* slot_tenant;     // [max_requests], -1 = closed
  int32_t* route;                 // [max_requests][n_layers][top_k]
  float* gate;                    // same shape: softmax probability of each selected module
  int32_t* err;                   // single flag word
  int n_layers, max_tenants, max_requests;
  int top_k, gating;
};

__host__ __device__ inline size_t adapter_index(int tenant, int layer, int module, int n_layers) {
  return ((size_t)tenant * n_layers + layer) * MILORA_NMOD + module;
}

// Where the four parts of one registered adapter sit inside its single pool allocation: A^T (rank x d1), B
// (rank x d2), then, when the operand images exist, the A image and the B image; every part starts on a 256-byte
// boundary.  Registration and the kernels that find the images from a job record's `At` use this one function.
constexpr int kImagePadMax = 64;   // largest padded rank that gets operand images
struct AdapterLayout {
  size_t off_b, off_a_img, off_b_img, total;
};
__host__ __device__ inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }
__host__ __device__ inline bool images_fit(int d1, int d2, int rank, size_t elem) {
  return elem == 2 && d1 % 64 == 0 && d2 % 128 == 0 && rank >= 1 && rank <= kImagePadMax;
}
__host__ __device__ inline AdapterLayout adapter_layout(int d1, int d2, int rank, size_t elem) {
  AdapterLayout L;
  const size_t rp = (size_t)((rank + 15) & ~15);
  const bool img = images_fit(d1, d2, rank, elem);
  L.off_b = align256((size_t)rank * d1 * elem);
  L.off_a_img = L.off_b + align256((size_t)rank * d2 * elem);
  L.off_b_img = L.off_a_img + (img ? align256((size_t)d1 * rp * 2) : 0);
  L.total = L.off_b_img + (img ? align256((size_t)d2 * rp * 2) : 0);
  return L;
}

// One layer of a multi-layer decode launch (apply_decode_stream.cu), as the kernel reads it.
constexpr int kMaxStreamLayers = 40;
struct StreamLayer {
  const int32_t* ws;                 // the layer's group block
  const void* X[MILORA_NMOD];        // nullptr: the module is skipped
  void* Y[MILORA_NMOD];
  int32_t off_header, off_mod_gather, off_gather, max_gather;   // int32 offsets into ws, capacity of the gather list
  int32_t T, job_base;               // rows of X / Y; first job slot of the layer in the launch's scratch arrays
};
static_assert(sizeof(StreamLayer) == 144, "StreamLayer is copied as 9 x 16 bytes");

// Pool behind the adapter and router copies: 64 MB (or larger) cudaMalloc chunks carved front to back, plus a list
// of blocks that were given back (a tenant that left, an adapter registered again at another rank), which
// allocations look through first.  Blocks are not merged; a server that churns tenants of a few sizes reuses them.
struct Arena {
  struct Chunk { char* base; size_t size, used; };
  struct Block { char* base; size_t size; };
  std::vector<Chunk> chunks;
  std::vector<Block> free_blocks;
  void* alloc(size_t bytes, cudaError_t* err);
  void give_back(void* p, size_t bytes);
  size_t bytes_in_use() const;      // carved bytes minus bytes on the free list
  void release();
};

}  // namespace milora

struct milora_ctx {
  milora_model_desc desc;
  int device;
  int sm_count;
  size_t elem;                                  // bytes per element of the context dtype
  std::vector<milora::AdapterEntry> h_adapters; // host mirrors
  std::vector<milora::RouterEntry> h_routers;
  std::vector<int32_t> h_slot_tenant;
  std::vector<size_t> adapter_bytes;            // pool bytes behind each adapter entry (for reuse)
  std::vector<size_t> router_bytes;
  size_t adapters_dirty_lo, adapters_dirty_hi;  // host-mirror ranges not yet uploaded
  size_t routers_dirty_lo, routers_dirty_hi;
  size_t slots_dirty_lo, slots_dirty_hi;
  milora::AdapterEntry* d_adapters;
  milora::RouterEntry* d_routers;
  int32_t* d_slot_tenant;
  int32_t* d_route;
  float* d_gate;
  int32_t* d_err;
  float* d_scratch;                             // router partial sums
  size_t scratch_floats;
  int32_t* d_counters;                          // router completion counters, one per prompt
  size_t n_counters;
  float* d_vscratch;                            // prefill: fp32 partial x.A products [k-split][T][rank_pad]
  size_t vscratch_floats;
  float* d_dsplit;                              // two-kernel decode path: unit counters (64 words), then v [jobs][rows][rank]
  size_t dsplit_floats;
  bool dsplit_dirty;                            // counters must be cleared before the next launch pair
  int dsplit_occ_s, dsplit_occ_e;               // resident CTAs per SM of its two kernels (0 = not asked yet)
  int decode_path;                              // milora_decode_path
  int n_routers_whole_row;                      // registered routers that pool by last token or self-attention
  bool route_bulk_attr_set;
  // persistent multi-layer decode kernel (apply_decode_stream.cu)
  void* d_stream;                               // control words, job states, v fragments, partial sums
  size_t stream_jobs_cap, stream_frag_bytes, stream_part_bytes;   // what d_stream is laid out for
  bool stream_dirty;                            // job states must be cleared before the next launch
  bool stream_attr_set;
  uint32_t stream_epoch;                        // tag of the last launch (marks the fragments it wrote)
  int stream_unit_stages;                       // stages per unit; 0 = chosen from the batch size
  void* d_stream_layers;                        // layer records of a multi-layer launch
  void* h_stream_stage;                         // pinned: four staging copies of those records
  cudaEvent_t stream_stage_ev[4];
  int stream_stage_next, stream_layers_cached;
  void* d_lin;                                  // fused projection: V piece images and per-row-block piece lists
  size_t lin_bytes;
  cudaStream_t copy_stream;                     // milora_step_host: device-to-host copies run beside the uploads
  cudaEvent_t ev_site[MILORA_NMOD];             // "module m is done" / "all copies back are done"
  cudaEvent_t ev_done;
  bool copy_ready;
  std::vector<int32_t> h_route_copy;            // milora_step_host: the route table as the host read it back
  milora::Arena arena;
  std::string cuda_error;
};

namespace milora {

milora_status cuda_fail(milora_ctx* ctx, cudaError_t e, const char* where);
#define MILORA_CUDA(ctx, call)                                        \
  do {                                                                \
    cudaError_t e__ = (call);                                         \
    if (e__ != cudaSuccess) return milora::cuda_fail((ctx), e__, #call); \
  } while (0)

// Uploads dirty ranges of the host mirrors on `stream`; called by every compute entry point.
milora_status sync_tables(milora_ctx* ctx, cudaStream_t stream);
DeviceTables device_tables(const milora_ctx* ctx);
void module_dims(const milora_model_desc& d, int module, int* d1, int* d2);
milora_group_layout_t group_layout(int n_seq, int T, int top_k);
inline int top_k_of(const milora_ctx* ctx) { return ctx->desc.top_k < 1 ? 1 : ctx->desc.top_k; }

// ---- programmatic dependent launch ---------------------------------------------------------------
// Every hot-path kernel is launched with the programmatic-stream-serialization attribute: it may start
// while the kernel before it on the stream is still draining, sets up its shared memory, barriers and
// tensor memory, and calls pdl_wait() before its first access to global memory (the wait returns once
// the preceding grid has completed and its writes are visible).  pdl_launch_dependents() at the top lets
// the kernel after it do the same.  Every CTA calls pdl_wait() before it can return, so completion of a
// grid implies completion of everything before it on the stream.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <class Args>
inline cudaError_t launch_pdl(void (*kernel)(Args), dim3 grid, dim3 block, size_t smem, cudaStream_t s, const Args& args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args);
}
#endif

// kernels (defined in their own .cu files)
milora_status launch_repack_adapter(milora_ctx* ctx, const void* A, const void* B, void* At, void* Bout, int d1, int d2,
                                    int rank, cudaStream_t s);
milora_status launch_repack_router(milora_ctx* ctx, const void* Wr, void* Wt, int d, cudaStream_t s);
milora_status launch_route(milora_ctx* ctx, int layer, const void* H, const int32_t* cu, const int32_t* seq_slot, int P,
                           int T_total, float* logits_out, float* probs_out, cudaStream_t s);
milora_status launch_route_static(milora_ctx* ctx, int layer, const void* H, const int32_t* cu, const int32_t* seq_slot,
                                  int P, int T_total, float* logits_out, float* probs_out, cudaStream_t s);
milora_status launch_group(milora_ctx* ctx, int layer_begin, int n_layers, const int32_t* cu, const int32_t* seq_slot,
                           int n_seq, int T, int32_t* ws, size_t ws_stride, cudaStream_t s);

struct ApplySite {
  int module;
  const void* X;
  void* Y;
  int d1, d2;
};
constexpr int kMaxSites = MILORA_NMOD;
struct ApplySites {
  ApplySite site[kMaxSites];
  int n;
};
// Generic SIMT path (any dtype, any shape): gathered rows (decode) or dense tiles (prefill).
milora_status launch_apply_generic(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                   bool dense, cudaStream_t s);
// bf16 decode path: one cluster of CTAs per gather job, bulk-copy staging, DSMEM reduction.
// Returns MILORA_E_SHAPE when shapes or alignment do not fit it (the caller then uses the generic path).
milora_status launch_apply_decode_bf16(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                       cudaStream_t s);

// bf16 decode path as two streaming kernels (shrink over whole rows of A^T, expand over column slices of B) that
// take equally sized units from a counter; v goes through a scratch buffer of the context.  Same convention.
milora_status launch_apply_decode_split(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                        cudaStream_t s);

// bf16 decode path as one persistent launch over any number of layers (operand images, bulk-copy rings).
// `layers` is a host array whose job_base fields the call fills in.  Same MILORA_E_SHAPE convention.
bool decode_stream_supported(const milora_ctx* ctx);
milora_status launch_apply_decode_stream(milora_ctx* ctx, StreamLayer* layers, int n_layers, int n_seq_hint,
                                         cudaStream_t s);

// bf16 prefill path: tcgen05 shrink and expand kernels over the dense tiles (same MILORA_E_SHAPE convention),
// and the registration-time packing of the operand images they read.
milora_status launch_apply_prefill_bf16(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                        cudaStream_t s);
// bf16 fused projection Y = X . W + b + LoRA term of the routed dense tiles (same MILORA_E_SHAPE convention).
milora_status launch_linear_prefill_bf16(milora_ctx* ctx, int layer, int module, const void* X, const void* Wt,
                                         const void* bias, void* Y, const milora_groups* g, cudaStream_t s);
bool prefill_images_supported(const milora_ctx* ctx, int d1, int d2, int rank);
size_t prefill_image_bytes(int d, int rank);
milora_status launch_pack_images(milora_ctx* ctx, const void* At, const void* B, void* At_img, void* B_img, int d1, int d2,
                                 int rank, cudaStream_t s);

}  // namespace milora
