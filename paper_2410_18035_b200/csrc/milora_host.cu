// Host side of libmilora: context, adapter / router / slot tables, argument validation.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "milora_internal.h"

namespace milora {

milora_status cuda_fail(milora_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) {
    ctx->cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " at " + where;
  }
  cudaGetLastError();  // clear the sticky-free error state
  return MILORA_E_CUDA;
}

void* Arena::alloc(size_t bytes, cudaError_t* err) {
  *err = cudaSuccess;
  bytes = (bytes + 255) & ~size_t(255);
  // first fit among the blocks that were given back; what is left of a larger block stays on the list
  for (size_t i = 0; i < free_blocks.size(); ++i) {
    if (free_blocks[i].size >= bytes) {
      char* p = free_blocks[i].base;
      if (free_blocks[i].size == bytes) {
        free_blocks[i] = free_blocks.back();
        free_blocks.pop_back();
      } else {
        free_blocks[i].base += bytes;
        free_blocks[i].size -= bytes;
      }
      return p;
    }
  }
  for (auto& c : chunks) {
    if (c.size - c.used >= bytes) {
      void* p = c.base + c.used;
      c.used += bytes;
      return p;
    }
  }
  size_t sz = std::max(bytes, size_t(64) << 20);
  char* base = nullptr;
  *err = cudaMalloc(&base, sz);
  if (*err != cudaSuccess) return nullptr;
  chunks.push_back({base, sz, bytes});
  return base;
}

void Arena::give_back(void* p, size_t bytes) {
  bytes = (bytes + 255) & ~size_t(255);
  if (!p || bytes == 0) return;
  try {
    free_blocks.push_back({static_cast<char*>(p), bytes});
  } catch (...) {
    // the list could not grow: the block stays unused until the context is destroyed
  }
}

size_t Arena::bytes_in_use() const {
  size_t n = 0;
  for (const auto& c : chunks) n += c.used;
  for (const auto& b : free_blocks) n -= b.size;
  return n;
}

void Arena::release() {
  for (auto& c : chunks) cudaFree(c.base);
  chunks.clear();
  free_blocks.clear();
}

void module_dims(const milora_model_desc& d, int module, int* d1, int* d2) {
  switch (module) {
    case MILORA_Q:
    case MILORA_O: *d1 = d.d_model; *d2 = d.d_model; break;
    case MILORA_K:
    case MILORA_V: *d1 = d.d_model; *d2 = d.d_kv; break;
    case MILORA_GATE:
    case MILORA_UP: *d1 = d.d_model; *d2 = d.d_ff; break;
    default: *d1 = d.d_ff; *d2 = d.d_model; break;
  }
}

static size_t round4(size_t v) { return (v + 3) & ~size_t(3); }

// Sizes for `top_k` selected modules per sequence: a token may sit in up to top_k buckets.
milora_group_layout_t group_layout(int n_seq, int T, int top_k) {
  milora_group_layout_t L;
  size_t o = 0;
  const size_t k = top_k < 1 ? 1 : (size_t)top_k;
  const size_t n_ent = (size_t)n_seq * k, TT = (size_t)T * k;
  L.header = o; o += kHeaderInts;
  L.mod_offset = o; o += 8;
  L.mod_tile_offset = o; o += 8;
  L.mod_gather_offset = o; o += 8;
  L.seg_key = o; o += round4(n_ent);
  L.seg_offset = o; o += round4(n_ent + 1);
  L.perm = o; o += round4(TT);
  L.max_tiles = (int)(TT / kTileRows + n_ent);
  L.tiles = o; o += (size_t)L.max_tiles * kJobInts;
  L.gather_rows = o; o += round4(2 * TT);      // row and sequence of every gathered (token, module) pair
  // gathered rows belong to sequences shorter than kLongSeq, so there are at most (kLongSeq - 1) per entry
  L.max_gather = (int)(std::min(TT, (size_t)(kLongSeq - 1) * n_ent) / kGatherRows + n_ent + 1);
  L.gather = o; o += (size_t)L.max_gather * kJobInts;
  L.seq_tile = o; o += (size_t)n_seq * 8;
  L.total = round4(o);
  return L;
}

DeviceTables device_tables(const milora_ctx* ctx) {
  DeviceTables t;
  t.adapters = ctx->d_adapters;
  t.routers = ctx->d_routers;
  t.slot_tenant = ctx->d_slot_tenant;
  t.route = ctx->d_route;
  t.gate = ctx->d_gate;
  t.top_k = top_k_of(ctx);
  t.gating = ctx->desc.gate;
  t.err = ctx->d_err;
  t.n_layers = ctx->desc.n_layers;
  t.max_tenants = ctx->desc.max_tenants;
  t.max_requests = ctx->desc.max_requests;
  return t;
}

template <class T>
static milora_status upload_range(milora_ctx* ctx, T* dev, const std::vector<T>& host, size_t& lo, size_t& hi,
                                  cudaStream_t s) {
  if (lo < hi) {
    MILORA_CUDA(ctx, cudaMemcpyAsync(dev + lo, host.data() + lo, (hi - lo) * sizeof(T), cudaMemcpyHostToDevice, s));
    // The source is pageable memory that the next registration may change: wait until it is consumed.
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  }
  lo = host.size();
  hi = 0;
  return MILORA_OK;
}

milora_status sync_tables(milora_ctx* ctx, cudaStream_t s) {
  milora_status st;
  if ((st = upload_range(ctx, ctx->d_adapters, ctx->h_adapters, ctx->adapters_dirty_lo, ctx->adapters_dirty_hi, s)))
    return st;
  if ((st = upload_range(ctx, ctx->d_routers, ctx->h_routers, ctx->routers_dirty_lo, ctx->routers_dirty_hi, s)))
    return st;
  if ((st = upload_range(ctx, ctx->d_slot_tenant, ctx->h_slot_tenant, ctx->slots_dirty_lo, ctx->slots_dirty_hi, s)))
    return st;
  return MILORA_OK;
}

static void mark(size_t& lo, size_t& hi, size_t i) {
  lo = std::min(lo, i);
  hi = std::max(hi, i + 1);
}

static cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

}  // namespace milora

using namespace milora;

extern "C" {

const char* milora_status_string(milora_status s) {
  switch (s) {
    case MILORA_OK: return "ok";
    case MILORA_E_ARG: return "invalid argument";
    case MILORA_E_SHAPE: return "unsupported shape";
    case MILORA_E_DTYPE: return "unsupported dtype";
    case MILORA_E_UNREGISTERED: return "not registered";
    case MILORA_E_CAPACITY: return "capacity exceeded";
    case MILORA_E_STATE: return "invalid state";
    case MILORA_E_CUDA: return "CUDA error";
    case MILORA_E_DEVICE_INDEX: return "a kernel skipped an out-of-range index";
  }
  return "unknown status";
}

const char* milora_last_cuda_error(const milora_ctx* ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

milora_status milora_create(const milora_model_desc* desc, milora_ctx** out) {
  if (!desc || !out) return MILORA_E_ARG;
  *out = nullptr;
  if (desc->dtype != MILORA_F32 && desc->dtype != MILORA_BF16) return MILORA_E_DTYPE;
  if (desc->n_layers < 1 || desc->d_model < 1 || desc->d_ff < 1 || desc->d_kv < 1) return MILORA_E_SHAPE;
  {
    // every row of every matrix must start on a 16-byte boundary (128-bit loads, bulk copies)
    const int vec = desc->dtype == MILORA_F32 ? 4 : 8;
    if (desc->d_model % vec || desc->d_ff % vec || desc->d_kv % vec) return MILORA_E_SHAPE;
  }
  if (desc->max_rank < 1 || desc->max_rank > 256) return MILORA_E_CAPACITY;
  if (desc->max_tenants < 1 || desc->max_requests < 1) return MILORA_E_CAPACITY;
  if ((long long)desc->max_tenants * MILORA_NMOD > (1ll << 30)) return MILORA_E_CAPACITY;
  if (desc->top_k < 0 || desc->top_k > MILORA_NMOD) return MILORA_E_ARG;
  if (desc->gate != MILORA_GATE_NONE && desc->gate != MILORA_GATE_PROB) return MILORA_E_ARG;
  milora_ctx* ctx = new (std::nothrow) milora_ctx();
  if (!ctx) return MILORA_E_CAPACITY;
  ctx->desc = *desc;
  ctx->elem = desc->dtype == MILORA_F32 ? 4 : 2;
  ctx->d_adapters = nullptr; ctx->d_routers = nullptr; ctx->d_slot_tenant = nullptr; ctx->d_route = nullptr;
  ctx->d_gate = nullptr;
  ctx->d_err = nullptr; ctx->d_scratch = nullptr; ctx->scratch_floats = 0; ctx->d_counters = nullptr;
  ctx->d_vscratch = nullptr; ctx->vscratch_floats = 0;
  ctx->d_lin = nullptr; ctx->lin_bytes = 0;
  ctx->d_dsplit = nullptr; ctx->dsplit_floats = 0; ctx->dsplit_dirty = true;
  ctx->dsplit_occ_s = 0; ctx->dsplit_occ_e = 0; ctx->decode_path = MILORA_DECODE_AUTO;
  ctx->n_routers_whole_row = 0; ctx->route_bulk_attr_set = false;
  ctx->copy_stream = nullptr; ctx->ev_done = nullptr; ctx->copy_ready = false;
  ctx->d_stream = nullptr; ctx->stream_jobs_cap = 0; ctx->stream_frag_bytes = 0; ctx->stream_part_bytes = 0;
  ctx->stream_dirty = true; ctx->stream_attr_set = false; ctx->stream_epoch = 0; ctx->stream_unit_stages = 0;
  ctx->d_stream_layers = nullptr; ctx->h_stream_stage = nullptr; ctx->stream_stage_next = 0; ctx->stream_layers_cached = 0;
  for (int i = 0; i < 4; ++i) ctx->stream_stage_ev[i] = nullptr;
  for (int m = 0; m < MILORA_NMOD; ++m) ctx->ev_site[m] = nullptr;
  ctx->n_counters = 0;
  milora_status st = MILORA_OK;
  auto fail = [&](milora_status s) { milora_destroy(ctx); return s; };
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e != cudaSuccess) { st = cuda_fail(ctx, e, "cudaGetDevice"); return fail(st); }
  e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e != cudaSuccess) { st = cuda_fail(ctx, e, "cudaDeviceGetAttribute"); return fail(st); }
  size_t n_ad = (size_t)desc->max_tenants * desc->n_layers * MILORA_NMOD;
  size_t n_rt = (size_t)desc->max_tenants * desc->n_layers;
  try {
    AdapterEntry a0;
    std::memset(&a0, 0, sizeof(a0));
    ctx->h_adapters.assign(n_ad, a0);
    RouterEntry r0;
    std::memset(&r0, 0, sizeof(r0));
    ctx->h_routers.assign(n_rt, r0);
    ctx->h_slot_tenant.assign(desc->max_requests, -1);
    ctx->adapter_bytes.assign(n_ad, 0);
    ctx->router_bytes.assign(n_rt, 0);
  } catch (...) {
    return fail(MILORA_E_CAPACITY);
  }
  ctx->adapters_dirty_lo = 0; ctx->adapters_dirty_hi = n_ad;
  ctx->routers_dirty_lo = 0; ctx->routers_dirty_hi = n_rt;
  ctx->slots_dirty_lo = 0; ctx->slots_dirty_hi = desc->max_requests;
  size_t route_bytes = (size_t)desc->max_requests * desc->n_layers * top_k_of(ctx) * sizeof(int32_t);
#define CREATE_CUDA(call)                                            \
  do {                                                               \
    cudaError_t e__ = (call);                                        \
    if (e__ != cudaSuccess) return fail(cuda_fail(ctx, e__, #call)); \
  } while (0)
  CREATE_CUDA(cudaMalloc(&ctx->d_adapters, n_ad * sizeof(AdapterEntry)));
  CREATE_CUDA(cudaMalloc(&ctx->d_routers, n_rt * sizeof(RouterEntry)));
  CREATE_CUDA(cudaMalloc(&ctx->d_slot_tenant, desc->max_requests * sizeof(int32_t)));
  CREATE_CUDA(cudaMalloc(&ctx->d_route, route_bytes));
  CREATE_CUDA(cudaMalloc(&ctx->d_gate, route_bytes));
  CREATE_CUDA(cudaMalloc(&ctx->d_err, 256));
  CREATE_CUDA(cudaMemset(ctx->d_route, 0xFF, route_bytes));
  CREATE_CUDA(cudaMemset(ctx->d_gate, 0, route_bytes));
  CREATE_CUDA(cudaMemset(ctx->d_err, 0, 256));
  st = sync_tables(ctx, nullptr);
  if (st != MILORA_OK) return fail(st);
  CREATE_CUDA(cudaDeviceSynchronize());
#undef CREATE_CUDA
  *out = ctx;
  return MILORA_OK;
}

milora_status milora_destroy(milora_ctx* ctx) {
  if (!ctx) return MILORA_OK;
  cudaFree(ctx->d_adapters);
  cudaFree(ctx->d_routers);
  cudaFree(ctx->d_slot_tenant);
  cudaFree(ctx->d_route);
  cudaFree(ctx->d_gate);
  cudaFree(ctx->d_err);
  cudaFree(ctx->d_scratch);
  cudaFree(ctx->d_counters);
  cudaFree(ctx->d_vscratch);
  cudaFree(ctx->d_lin);
  cudaFree(ctx->d_dsplit);
  cudaFree(ctx->d_stream);
  cudaFree(ctx->d_stream_layers);
  if (ctx->h_stream_stage) cudaFreeHost(ctx->h_stream_stage);
  for (int i = 0; i < 4; ++i)
    if (ctx->stream_stage_ev[i]) cudaEventDestroy(ctx->stream_stage_ev[i]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->ev_done) cudaEventDestroy(ctx->ev_done);
  for (int m = 0; m < MILORA_NMOD; ++m)
    if (ctx->ev_site[m]) cudaEventDestroy(ctx->ev_site[m]);
  ctx->arena.release();
  delete ctx;
  return MILORA_OK;
}

milora_status milora_module_dims(const milora_ctx* ctx, int module, int* d1, int* d2) {
  if (!ctx || !d1 || !d2 || module < 0 || module >= MILORA_NMOD) return MILORA_E_ARG;
  module_dims(ctx->desc, module, d1, d2);
  return MILORA_OK;
}

milora_status milora_register_adapter(milora_ctx* ctx, int tenant, int layer, int module, int rank, float scale,
                                      const void* A_dev, const void* B_dev, void* stream) {
  if (!ctx || !A_dev || !B_dev) return MILORA_E_ARG;
  if (tenant < 0 || tenant >= ctx->desc.max_tenants || layer < 0 || layer >= ctx->desc.n_layers || module < 0 ||
      module >= MILORA_NMOD)
    return MILORA_E_ARG;
  if (rank < 1) return MILORA_E_ARG;
  if (rank > ctx->desc.max_rank) return MILORA_E_CAPACITY;
  int d1, d2;
  module_dims(ctx->desc, module, &d1, &d2);
  size_t idx = adapter_index(tenant, layer, module, ctx->desc.n_layers);
  // tensor-core operand images (bf16 contexts, dimensions that fit the tiled kernels) follow A^T and B in the
  // same allocation; adapter_layout is also what the kernels use to find them from a job record
  const bool images = prefill_images_supported(ctx, d1, d2, rank);
  const AdapterLayout lay = adapter_layout(d1, d2, rank, ctx->elem);
  if (images != images_fit(d1, d2, rank, ctx->elem)) return MILORA_E_STATE;
  const size_t total = lay.total;
  AdapterEntry& ent = ctx->h_adapters[idx];
  void* store = const_cast<void*>(ent.At);
  if (!store || ctx->adapter_bytes[idx] != total) {
    cudaError_t e;
    if (store) ctx->arena.give_back(store, ctx->adapter_bytes[idx]);      // another rank than before: the old block is free
    ent.At = nullptr;
    ctx->adapter_bytes[idx] = 0;
    store = ctx->arena.alloc(total, &e);
    if (!store) return cuda_fail(ctx, e, "adapter pool cudaMalloc");
    ctx->adapter_bytes[idx] = total;
  }
  void* At = store;
  void* Bs = static_cast<char*>(store) + lay.off_b;
  void* Ai = images ? static_cast<char*>(store) + lay.off_a_img : nullptr;
  void* Bi = images ? static_cast<char*>(store) + lay.off_b_img : nullptr;
  milora_status st = launch_repack_adapter(ctx, A_dev, B_dev, At, Bs, d1, d2, rank, as_stream(stream));
  if (st != MILORA_OK) return st;
  if (images) {
    st = launch_pack_images(ctx, At, Bs, Ai, Bi, d1, d2, rank, as_stream(stream));
    if (st != MILORA_OK) return st;
  }
  ent.At = At;
  ent.B = Bs;
  ent.At_img = Ai;
  ent.B_img = Bi;
  ent.rank = rank;
  ent.rank_pad = (rank + 15) & ~15;
  ent.scale = scale;
  mark(ctx->adapters_dirty_lo, ctx->adapters_dirty_hi, idx);
  return MILORA_OK;
}

milora_status milora_register_router(milora_ctx* ctx, int tenant, int layer, const void* Wr_dev,
                                     const float* bias_dev, milora_pool pool, const void* Wsa_dev, milora_act act,
                                     const float* coef_host, int n_a, int n_b, void* stream) {
  if (!ctx || !Wr_dev) return MILORA_E_ARG;
  if (tenant < 0 || tenant >= ctx->desc.max_tenants || layer < 0 || layer >= ctx->desc.n_layers) return MILORA_E_ARG;
  if (pool < MILORA_POOL_MEAN || pool > MILORA_POOL_SELFATTN) return MILORA_E_ARG;
  if (act < MILORA_ACT_TANH || act > MILORA_ACT_RATIONAL) return MILORA_E_ARG;
  if (pool == MILORA_POOL_SELFATTN && !Wsa_dev) return MILORA_E_ARG;
  if (act == MILORA_ACT_RATIONAL) {
    if (!coef_host || n_a < 1 || n_b < 0 || n_a + n_b > MILORA_MAX_RATIONAL_COEF) return MILORA_E_ARG;
  } else {
    n_a = n_b = 0;
  }
  cudaStream_t s = as_stream(stream);
  size_t idx = (size_t)tenant * ctx->desc.n_layers + layer;
  int d = ctx->desc.d_model;
  size_t bytes_w = ((size_t)MILORA_NMOD * d * ctx->elem + 255) & ~size_t(255);
  size_t bytes_sa = ((size_t)d * ctx->elem + 255) & ~size_t(255);
  RouterEntry& ent = ctx->h_routers[idx];
  auto whole_row = [](const RouterEntry& r) {
    return r.W != nullptr && (r.pool == MILORA_POOL_LAST || r.pool == MILORA_POOL_SELFATTN);
  };
  if (whole_row(ent)) --ctx->n_routers_whole_row;        // replaced below
  void* store = const_cast<void*>(ent.W);
  if (!store || ctx->router_bytes[idx] != bytes_w + bytes_sa) {
    cudaError_t e;
    if (store) ctx->arena.give_back(store, ctx->router_bytes[idx]);
    ent.W = nullptr;
    ctx->router_bytes[idx] = 0;
    store = ctx->arena.alloc(bytes_w + bytes_sa, &e);
    if (!store) return cuda_fail(ctx, e, "router pool cudaMalloc");
    ctx->router_bytes[idx] = bytes_w + bytes_sa;
  }
  void* Wt = store;
  void* Wsa = static_cast<char*>(store) + bytes_w;
  milora_status st = launch_repack_router(ctx, Wr_dev, Wt, d, s);
  if (st != MILORA_OK) return st;
  if (Wsa_dev) MILORA_CUDA(ctx, cudaMemcpyAsync(Wsa, Wsa_dev, (size_t)d * ctx->elem, cudaMemcpyDeviceToDevice, s));
  std::memset(ent.bias, 0, sizeof(ent.bias));
  if (bias_dev) {
    MILORA_CUDA(ctx, cudaMemcpyAsync(ent.bias, bias_dev, MILORA_NMOD * sizeof(float), cudaMemcpyDeviceToHost, s));
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  }
  std::memset(ent.coef, 0, sizeof(ent.coef));
  for (int i = 0; i < n_a + n_b; ++i) ent.coef[i] = coef_host[i];
  ent.W = Wt;
  ent.Wsa = Wsa_dev ? Wsa : nullptr;
  ent.pool = pool;
  ent.act = act;
  ent.n_a = n_a;
  ent.n_b = n_b;
  if (whole_row(ent)) ++ctx->n_routers_whole_row;
  mark(ctx->routers_dirty_lo, ctx->routers_dirty_hi, idx);
  return MILORA_OK;
}

milora_status milora_unregister_tenant(milora_ctx* ctx, int tenant) {
  if (!ctx || tenant < 0 || tenant >= ctx->desc.max_tenants) return MILORA_E_ARG;
  for (int t : ctx->h_slot_tenant)
    if (t == tenant) return MILORA_E_STATE;
  int L = ctx->desc.n_layers;
  for (int l = 0; l < L; ++l) {
    for (int m = 0; m < MILORA_NMOD; ++m) {
      size_t idx = adapter_index(tenant, l, m, L);
      // the copies go back to the pool (the caller has made sure nothing that reads them is still running)
      AdapterEntry& ent = ctx->h_adapters[idx];
      ctx->arena.give_back(const_cast<void*>(ent.At), ctx->adapter_bytes[idx]);
      ctx->adapter_bytes[idx] = 0;
      std::memset(&ent, 0, sizeof(ent));
      mark(ctx->adapters_dirty_lo, ctx->adapters_dirty_hi, idx);
    }
    size_t r = (size_t)tenant * L + l;
    RouterEntry& rt = ctx->h_routers[r];
    if (rt.W != nullptr && (rt.pool == MILORA_POOL_LAST || rt.pool == MILORA_POOL_SELFATTN)) --ctx->n_routers_whole_row;
    ctx->arena.give_back(const_cast<void*>(rt.W), ctx->router_bytes[r]);
    ctx->router_bytes[r] = 0;
    std::memset(&rt, 0, sizeof(rt));
    rt.pool = -1;
    mark(ctx->routers_dirty_lo, ctx->routers_dirty_hi, r);
  }
  return MILORA_OK;
}

milora_status milora_resident_bytes(const milora_ctx* ctx, size_t* adapter_pool_bytes) {
  if (!ctx || !adapter_pool_bytes) return MILORA_E_ARG;
  *adapter_pool_bytes = ctx->arena.bytes_in_use();
  return MILORA_OK;
}

milora_status milora_request_open(milora_ctx* ctx, int slot, int tenant) {
  if (!ctx || slot < 0 || slot >= ctx->desc.max_requests || tenant < 0 || tenant >= ctx->desc.max_tenants)
    return MILORA_E_ARG;
  if (ctx->h_slot_tenant[slot] >= 0) return MILORA_E_STATE;
  // The route row of a freshly opened slot must read "not routed".
  // The slot is closed, so no kernel in flight reads this row; the reset is finished before returning.
  const size_t row = (size_t)ctx->desc.n_layers * top_k_of(ctx);
  MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_route + (size_t)slot * row, 0xFF, row * sizeof(int32_t), nullptr));
  MILORA_CUDA(ctx, cudaStreamSynchronize(nullptr));
  ctx->h_slot_tenant[slot] = tenant;
  mark(ctx->slots_dirty_lo, ctx->slots_dirty_hi, (size_t)slot);
  return MILORA_OK;
}

milora_status milora_request_close(milora_ctx* ctx, int slot) {
  if (!ctx || slot < 0 || slot >= ctx->desc.max_requests) return MILORA_E_ARG;
  if (ctx->h_slot_tenant[slot] < 0) return MILORA_E_STATE;
  ctx->h_slot_tenant[slot] = -1;
  mark(ctx->slots_dirty_lo, ctx->slots_dirty_hi, (size_t)slot);
  return MILORA_OK;
}

milora_status milora_route(milora_ctx* ctx, int layer, const void* H_dev, const int32_t* cu_seqlens_dev,
                           const int32_t* seq_slot_dev, int P, int T_total, float* logits_out_dev,
                           float* probs_out_dev, void* stream) {
  if (!ctx) return MILORA_E_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers || P < 0 || T_total < 0) return MILORA_E_ARG;
  if (P > kMaxSeq) return MILORA_E_CAPACITY;
  if (P == 0) return MILORA_OK;
  if (!cu_seqlens_dev || !seq_slot_dev || (T_total > 0 && !H_dev)) return MILORA_E_ARG;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);
  if (st != MILORA_OK) return st;
  return launch_route(ctx, layer, H_dev, cu_seqlens_dev, seq_slot_dev, P, T_total, logits_out_dev, probs_out_dev, s);
}

milora_status milora_route_static(milora_ctx* ctx, int layer, const void* H_dev, const int32_t* cu_seqlens_dev,
                                  const int32_t* seq_slot_dev, int P, int T_total, float* logits_out_dev,
                                  float* probs_out_dev, void* stream) {
  if (!ctx) return MILORA_E_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers || P < 0 || T_total < 0) return MILORA_E_ARG;
  if (P > kMaxSeq) return MILORA_E_CAPACITY;
  if (P == 0) return MILORA_OK;
  if (!cu_seqlens_dev || !seq_slot_dev || (T_total > 0 && !H_dev)) return MILORA_E_ARG;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);   // copies pending table updates; allocates nothing
  if (st != MILORA_OK) return st;
  return launch_route_static(ctx, layer, H_dev, cu_seqlens_dev, seq_slot_dev, P, T_total, logits_out_dev,
                             probs_out_dev, s);
}

milora_status milora_route_table(const milora_ctx* ctx, const int32_t** table_dev) {
  if (!ctx || !table_dev) return MILORA_E_ARG;
  *table_dev = ctx->d_route;
  return MILORA_OK;
}

milora_status milora_route_table_read(milora_ctx* ctx, int slot_begin, int n_slots, int32_t* rows_host, void* stream) {
  if (!ctx || !rows_host || slot_begin < 0 || n_slots < 0 || slot_begin + n_slots > ctx->desc.max_requests)
    return MILORA_E_ARG;
  if (n_slots == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  size_t L = (size_t)ctx->desc.n_layers * top_k_of(ctx);
  MILORA_CUDA(ctx, cudaMemcpyAsync(rows_host, ctx->d_route + (size_t)slot_begin * L, (size_t)n_slots * L * sizeof(int32_t),
                                   cudaMemcpyDeviceToHost, s));
  MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  return MILORA_OK;
}

milora_status milora_gate_table_read(milora_ctx* ctx, int slot_begin, int n_slots, float* rows_host, void* stream) {
  if (!ctx || !rows_host || slot_begin < 0 || n_slots < 0 || slot_begin + n_slots > ctx->desc.max_requests)
    return MILORA_E_ARG;
  if (n_slots == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  size_t L = (size_t)ctx->desc.n_layers * top_k_of(ctx);
  MILORA_CUDA(ctx, cudaMemcpyAsync(rows_host, ctx->d_gate + (size_t)slot_begin * L, (size_t)n_slots * L * sizeof(float),
                                   cudaMemcpyDeviceToHost, s));
  MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  return MILORA_OK;
}

milora_status milora_gate_table_write(milora_ctx* ctx, int slot_begin, int n_slots, const float* rows_host,
                                      void* stream) {
  if (!ctx || !rows_host || slot_begin < 0 || n_slots < 0 || slot_begin + n_slots > ctx->desc.max_requests)
    return MILORA_E_ARG;
  if (n_slots == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  size_t L = (size_t)ctx->desc.n_layers * top_k_of(ctx);
  MILORA_CUDA(ctx, cudaMemcpyAsync(ctx->d_gate + (size_t)slot_begin * L, rows_host, (size_t)n_slots * L * sizeof(float),
                                   cudaMemcpyHostToDevice, s));
  MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  return MILORA_OK;
}

milora_status milora_route_table_write(milora_ctx* ctx, int slot_begin, int n_slots, const int32_t* rows_host,
                                       void* stream) {
  if (!ctx || !rows_host || slot_begin < 0 || n_slots < 0 || slot_begin + n_slots > ctx->desc.max_requests)
    return MILORA_E_ARG;
  size_t L = (size_t)ctx->desc.n_layers * top_k_of(ctx);
  for (size_t i = 0; i < (size_t)n_slots * L; ++i)
    if (rows_host[i] < -1 || rows_host[i] >= MILORA_NMOD) return MILORA_E_ARG;
  {
    // the modules selected for one (slot, layer) must be distinct: a module is applied at most once
    const size_t K = top_k_of(ctx);
    for (size_t c = 0; c < (size_t)n_slots * ctx->desc.n_layers; ++c) {
      unsigned seen = 0;
      for (size_t j = 0; j < K; ++j) {
        const int m = rows_host[c * K + j];
        if (m < 0) continue;
        if ((seen >> m) & 1u) return MILORA_E_ARG;
        seen |= 1u << m;
      }
    }
  }
  if (n_slots == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  MILORA_CUDA(ctx, cudaMemcpyAsync(ctx->d_route + (size_t)slot_begin * L, rows_host, (size_t)n_slots * L * sizeof(int32_t),
                                   cudaMemcpyHostToDevice, s));
  MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  return MILORA_OK;
}

milora_status milora_group_layout(const milora_ctx* ctx, int n_seq, int T, milora_group_layout_t* out) {
  if (!ctx || !out || n_seq < 0 || T < 0) return MILORA_E_ARG;
  if ((long long)n_seq * top_k_of(ctx) > kMaxSeq) return MILORA_E_CAPACITY;
  *out = group_layout(n_seq, T, top_k_of(ctx));
  return MILORA_OK;
}

milora_status milora_group(milora_ctx* ctx, int layer_begin, int n_layers, const int32_t* cu_seqlens_dev,
                           const int32_t* seq_slot_dev, int n_seq, int T, int32_t* ws_dev, size_t ws_stride,
                           void* stream) {
  if (!ctx || !ws_dev) return MILORA_E_ARG;
  if (layer_begin < 0 || n_layers < 1 || layer_begin + n_layers > ctx->desc.n_layers) return MILORA_E_ARG;
  if (n_seq < 0 || T < 0 || (n_seq > 0 && !seq_slot_dev)) return MILORA_E_ARG;
  if ((long long)n_seq * top_k_of(ctx) > kMaxSeq) return MILORA_E_CAPACITY;
  if (!cu_seqlens_dev && T != n_seq) return MILORA_E_ARG;
  milora_group_layout_t L = group_layout(n_seq, T, top_k_of(ctx));
  if (ws_stride < L.total || (ws_stride & 3) || (reinterpret_cast<uintptr_t>(ws_dev) & 15)) return MILORA_E_ARG;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);
  if (st != MILORA_OK) return st;
  return launch_group(ctx, layer_begin, n_layers, cu_seqlens_dev, seq_slot_dev, n_seq, T, ws_dev, ws_stride, s);
}

// AUTO: the two-kernel path once the work list has room for more than two jobs per SM (measured on the decode
// batch sweep: at 128 requests on 128 tenants the single launch is still 10 % faster, at 256 the pair is 12 %
// faster; 13B shapes at 256 requests: 29 %).
static milora_decode_path pick_decode_path(const milora_ctx* ctx, int n_seq, int T) {
  if (ctx->decode_path == MILORA_DECODE_STREAM && !decode_stream_supported(ctx)) return MILORA_DECODE_CLUSTER;
  if (ctx->decode_path != MILORA_DECODE_AUTO) return (milora_decode_path)ctx->decode_path;
  // One layer per call, measured (8B and 13B shapes, rank 16 and 32): up to 64 sequences the cluster kernel is the
  // quickest (12.9 against 15.7 us at 64), from 128 on the persistent kernel (20.1 against 21.6 us at 128, 30.2
  // against 34.2 at 256, 40.9 against 49.8 on the 13B step).
  if (n_seq >= 96 && decode_stream_supported(ctx)) return MILORA_DECODE_STREAM;
  const milora_group_layout_t lay = group_layout(n_seq, T, top_k_of(ctx));
  return lay.max_gather > 2 * ctx->sm_count ? MILORA_DECODE_SPLIT : MILORA_DECODE_CLUSTER;
}

milora_status milora_decode_path_for(const milora_ctx* ctx, int n_seq, int T, milora_decode_path* out) {
  if (!ctx || !out || n_seq < 0 || T < 0) return MILORA_E_ARG;
  *out = pick_decode_path(ctx, n_seq, T);
  return MILORA_OK;
}

// The part of a layer record that follows from the group block alone.
static StreamLayer stream_layer_of(const milora_ctx* ctx, const milora_groups* g) {
  StreamLayer L;
  std::memset(&L, 0, sizeof(L));
  const milora_group_layout_t lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  L.ws = g->ws_dev;
  L.off_header = (int32_t)lay.header;
  L.off_mod_gather = (int32_t)lay.mod_gather_offset;
  L.off_gather = (int32_t)lay.gather;
  L.max_gather = lay.max_gather;
  L.T = g->T;
  return L;
}

static milora_status apply_common(milora_ctx* ctx, int layer, int n_sites, const int* modules,
                                  const void* const* X_dev, void* const* Y_dev, const milora_groups* groups,
                                  bool dense, void* stream) {
  if (!ctx || !groups || !modules || !X_dev || !Y_dev) return MILORA_E_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return MILORA_E_ARG;
  if (n_sites < 1 || n_sites > kMaxSites) return MILORA_E_ARG;
  if (!groups->ws_dev || groups->n_seq < 0 || groups->T < 0 || (long long)groups->n_seq * top_k_of(ctx) > kMaxSeq)
    return MILORA_E_ARG;
  ApplySites sites;
  sites.n = n_sites;
  unsigned seen = 0;
  for (int i = 0; i < n_sites; ++i) {
    int m = modules[i];
    if (m < 0 || m >= MILORA_NMOD || (seen >> m & 1)) return MILORA_E_ARG;
    seen |= 1u << m;
    if (groups->T > 0 && (!X_dev[i] || !Y_dev[i])) return MILORA_E_ARG;
    sites.site[i].module = m;
    sites.site[i].X = X_dev[i];
    sites.site[i].Y = Y_dev[i];
    module_dims(ctx->desc, m, &sites.site[i].d1, &sites.site[i].d2);
  }
  if (groups->T == 0 || groups->n_seq == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);
  if (st != MILORA_OK) return st;
  if (ctx->desc.dtype == MILORA_BF16) {
    if (dense) {
      st = launch_apply_prefill_bf16(ctx, layer, sites, groups, s);
    } else {
      st = MILORA_E_SHAPE;
      const milora_decode_path path = pick_decode_path(ctx, groups->n_seq, groups->T);
      if (path == MILORA_DECODE_STREAM) {
        StreamLayer one = stream_layer_of(ctx, groups);
        bool aligned = true;
        for (int i = 0; i < sites.n; ++i) {
          one.X[sites.site[i].module] = sites.site[i].X;
          one.Y[sites.site[i].module] = sites.site[i].Y;
          aligned = aligned && !((reinterpret_cast<uintptr_t>(sites.site[i].X) | reinterpret_cast<uintptr_t>(sites.site[i].Y)) & 15);
        }
        if (aligned) st = launch_apply_decode_stream(ctx, &one, 1, groups->n_seq, s);
      } else if (path == MILORA_DECODE_SPLIT) {
        st = launch_apply_decode_split(ctx, layer, sites, groups, s);
      }
      if (st == MILORA_E_SHAPE) st = launch_apply_decode_bf16(ctx, layer, sites, groups, s);
    }
    if (st != MILORA_E_SHAPE) return st;     // MILORA_E_SHAPE: this batch does not fit the specialised kernel
  }
  return launch_apply_generic(ctx, layer, sites, groups, dense, s);
}

milora_status milora_set_decode_path(milora_ctx* ctx, milora_decode_path path) {
  if (!ctx) return MILORA_E_ARG;
  if (path != MILORA_DECODE_AUTO && path != MILORA_DECODE_CLUSTER && path != MILORA_DECODE_SPLIT &&
      path != MILORA_DECODE_STREAM)
    return MILORA_E_ARG;
  ctx->decode_path = (int)path;
  return MILORA_OK;
}

milora_status milora_set_decode_unit_stages(milora_ctx* ctx, int unit_stages) {
  if (!ctx || unit_stages < 0 || unit_stages > 64) return MILORA_E_ARG;
  ctx->stream_unit_stages = unit_stages;
  return MILORA_OK;
}

milora_status milora_apply_decode_layers(milora_ctx* ctx, const milora_decode_layer* layers, int n_layers, void* stream) {
  if (!ctx || n_layers < 0 || (n_layers > 0 && !layers)) return MILORA_E_ARG;
  if (n_layers == 0) return MILORA_OK;
  std::vector<StreamLayer> recs;
  std::vector<int> keep;
  try {
    recs.reserve(n_layers);
    keep.reserve(n_layers);
  } catch (...) {
    return MILORA_E_CAPACITY;
  }
  int n_seq_hint = 0;
  for (int i = 0; i < n_layers; ++i) {
    const milora_decode_layer& d = layers[i];
    if (d.layer < 0 || d.layer >= ctx->desc.n_layers) return MILORA_E_ARG;
    const milora_groups& g = d.groups;
    if (!g.ws_dev || g.n_seq < 0 || g.T < 0 || (long long)g.n_seq * top_k_of(ctx) > kMaxSeq) return MILORA_E_ARG;
    bool any = false;
    for (int m = 0; m < MILORA_NMOD; ++m) {
      if ((d.X_dev[m] == nullptr) != (d.Y_dev[m] == nullptr)) return MILORA_E_ARG;
      any = any || d.X_dev[m];
    }
    if (!any || g.T == 0 || g.n_seq == 0) continue;
    StreamLayer L = stream_layer_of(ctx, &g);
    for (int m = 0; m < MILORA_NMOD; ++m) {
      L.X[m] = d.X_dev[m];
      L.Y[m] = d.Y_dev[m];
    }
    recs.push_back(L);
    keep.push_back(i);
    n_seq_hint = std::max(n_seq_hint, g.n_seq);
  }
  if (recs.empty()) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);
  if (st != MILORA_OK) return st;
  bool aligned = true;
  for (const StreamLayer& L : recs)
    for (int m = 0; m < MILORA_NMOD; ++m)
      aligned = aligned && !((reinterpret_cast<uintptr_t>(L.X[m]) | reinterpret_cast<uintptr_t>(L.Y[m])) & 15);
  if (decode_stream_supported(ctx) && aligned && ctx->decode_path != MILORA_DECODE_CLUSTER &&
      ctx->decode_path != MILORA_DECODE_SPLIT) {
    st = launch_apply_decode_stream(ctx, recs.data(), (int)recs.size(), n_seq_hint, s);
    if (st != MILORA_E_SHAPE) return st;
  }
  // shapes, dtype or a forced kernel set that the persistent kernel does not cover: one call per layer
  for (int i : keep) {
    const milora_decode_layer& d = layers[i];
    int mods[MILORA_NMOD], n = 0;
    const void* X[MILORA_NMOD];
    void* Y[MILORA_NMOD];
    for (int m = 0; m < MILORA_NMOD; ++m)
      if (d.X_dev[m]) { mods[n] = m; X[n] = d.X_dev[m]; Y[n] = d.Y_dev[m]; ++n; }
    st = apply_common(ctx, d.layer, n, mods, X, Y, &d.groups, false, stream);
    if (st != MILORA_OK) return st;
  }
  return MILORA_OK;
}

milora_status milora_apply_decode(milora_ctx* ctx, int layer, int module, const void* X_dev, void* Y_dev,
                                  const milora_groups* groups, void* stream) {
  return apply_common(ctx, layer, 1, &module, &X_dev, &Y_dev, groups, false, stream);
}

milora_status milora_apply_prefill(milora_ctx* ctx, int layer, int module, const void* X_dev, void* Y_dev,
                                   const milora_groups* groups, void* stream) {
  return apply_common(ctx, layer, 1, &module, &X_dev, &Y_dev, groups, true, stream);
}

milora_status milora_apply_decode_multi(milora_ctx* ctx, int layer, int n_sites, const int* modules,
                                        const void* const* X_dev, void* const* Y_dev, const milora_groups* groups,
                                        void* stream) {
  return apply_common(ctx, layer, n_sites, modules, X_dev, Y_dev, groups, false, stream);
}

milora_status milora_apply_prefill_multi(milora_ctx* ctx, int layer, int n_sites, const int* modules,
                                         const void* const* X_dev, void* const* Y_dev, const milora_groups* groups,
                                         void* stream) {
  return apply_common(ctx, layer, n_sites, modules, X_dev, Y_dev, groups, true, stream);
}

milora_status milora_apply_prefill_shared(milora_ctx* ctx, int layer, int n_sites, const int* modules, const void* X_dev,
                                          void* const* Y_dev, const milora_groups* groups, void* stream) {
  if (!ctx || !modules || n_sites < 1 || n_sites > kMaxSites) return MILORA_E_ARG;
  const void* X[kMaxSites];
  int d1_first = 0;
  for (int i = 0; i < n_sites; ++i) {
    if (modules[i] < 0 || modules[i] >= MILORA_NMOD) return MILORA_E_ARG;
    int d1, d2;
    module_dims(ctx->desc, modules[i], &d1, &d2);
    if (i == 0) d1_first = d1;
    if (d1 != d1_first) return MILORA_E_ARG;      // modules that read one matrix have one input width
    X[i] = X_dev;
  }
  return apply_common(ctx, layer, n_sites, modules, X, Y_dev, groups, true, stream);
}

milora_status milora_linear_prefill(milora_ctx* ctx, int layer, int module, const void* X_dev, const void* Wt_dev,
                                    const void* bias_dev, void* Y_dev, const milora_groups* groups, void* stream) {
  if (!ctx || !groups || !X_dev || !Wt_dev || !Y_dev) return MILORA_E_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers || module < 0 || module >= MILORA_NMOD) return MILORA_E_ARG;
  if (!groups->ws_dev || groups->n_seq < 0 || groups->T < 0 || (long long)groups->n_seq * top_k_of(ctx) > kMaxSeq)
    return MILORA_E_ARG;
  if (groups->T == 0) return MILORA_OK;
  cudaStream_t s = as_stream(stream);
  milora_status st = sync_tables(ctx, s);
  if (st != MILORA_OK) return st;
  return launch_linear_prefill_bf16(ctx, layer, module, X_dev, Wt_dev, bias_dev, Y_dev, groups, s);
}

// ---- one step from host buffers ---------------------------------------------------------------------
namespace {
struct HostStepPlan {
  size_t H, cu_p, slot_p, cu_s, slot_s, ws, X[MILORA_NMOD], Y[MILORA_NMOD], total;
  size_t ws_stride;
  int T_p;
};
size_t up256(size_t v) { return (v + 255) & ~size_t(255); }

milora_status plan_host_step(const milora_ctx* ctx, const milora_host_step* st, HostStepPlan* pl) {
  if (!ctx || !st || !pl) return MILORA_E_ARG;
  if (st->layer < 0 || st->layer >= ctx->desc.n_layers) return MILORA_E_ARG;
  if (st->n_prompts < 0 || st->n_seq < 0 || st->T < 0) return MILORA_E_ARG;
  if (st->n_prompts > kMaxSeq || st->n_seq > kMaxSeq) return MILORA_E_CAPACITY;
  if (st->n_prompts > 0 && (!st->cu_prompts_host || !st->prompt_slot_host)) return MILORA_E_ARG;
  if (st->n_seq > 0 && (!st->cu_seq_host || !st->seq_slot_host)) return MILORA_E_ARG;
  pl->T_p = st->n_prompts > 0 ? st->cu_prompts_host[st->n_prompts] : 0;
  if (pl->T_p < 0 || (pl->T_p > 0 && !st->H_host)) return MILORA_E_ARG;
  size_t o = 0;
  pl->H = o; o += up256((size_t)pl->T_p * ctx->desc.d_model * ctx->elem);
  pl->cu_p = o; o += up256((size_t)(st->n_prompts + 1) * 4);
  pl->slot_p = o; o += up256((size_t)st->n_prompts * 4 + 4);
  pl->cu_s = o; o += up256((size_t)(st->n_seq + 1) * 4);
  pl->slot_s = o; o += up256((size_t)st->n_seq * 4 + 4);
  if ((long long)st->n_seq * top_k_of(ctx) > kMaxSeq) return MILORA_E_CAPACITY;
  pl->ws_stride = group_layout(st->n_seq, st->T, top_k_of(ctx)).total;
  pl->ws = o; o += up256(pl->ws_stride * 4);
  for (int m = 0; m < MILORA_NMOD; ++m) {
    pl->X[m] = pl->Y[m] = 0;
    if ((st->X_host[m] == nullptr) != (st->Y_host[m] == nullptr)) return MILORA_E_ARG;
    if (!st->X_host[m]) continue;
    int d1, d2;
    module_dims(ctx->desc, m, &d1, &d2);
    pl->X[m] = o; o += up256((size_t)st->T * d1 * ctx->elem);
    pl->Y[m] = o; o += up256((size_t)st->T * d2 * ctx->elem);
  }
  pl->total = o;
  return MILORA_OK;
}
}  // namespace

milora_status milora_step_host_workspace(const milora_ctx* ctx, const milora_host_step* step, size_t* bytes) {
  if (!bytes) return MILORA_E_ARG;
  HostStepPlan pl;
  milora_status st = plan_host_step(ctx, step, &pl);
  if (st != MILORA_OK) return st;
  *bytes = pl.total;
  return MILORA_OK;
}

milora_status milora_step_host(milora_ctx* ctx, const milora_host_step* step, void* workspace_dev,
                               size_t workspace_bytes, void* stream) {
  HostStepPlan pl;
  milora_status st = plan_host_step(ctx, step, &pl);
  if (st != MILORA_OK) return st;
  if (!workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255) || workspace_bytes < pl.total)
    return MILORA_E_ARG;
  char* w = static_cast<char*>(workspace_dev);
  cudaStream_t s = as_stream(stream);
  const size_t e = ctx->elem;
  auto h2d = [&](size_t off, const void* src, size_t bytes) -> cudaError_t {
    return bytes ? cudaMemcpyAsync(w + off, src, bytes, cudaMemcpyHostToDevice, s) : cudaSuccess;
  };
  // inputs
  MILORA_CUDA(ctx, h2d(pl.H, step->H_host, (size_t)pl.T_p * ctx->desc.d_model * e));
  if (step->n_prompts > 0) {
    MILORA_CUDA(ctx, h2d(pl.cu_p, step->cu_prompts_host, (size_t)(step->n_prompts + 1) * 4));
    MILORA_CUDA(ctx, h2d(pl.slot_p, step->prompt_slot_host, (size_t)step->n_prompts * 4));
  }
  if (step->n_seq > 0) {
    MILORA_CUDA(ctx, h2d(pl.cu_s, step->cu_seq_host, (size_t)(step->n_seq + 1) * 4));
    MILORA_CUDA(ctx, h2d(pl.slot_s, step->seq_slot_host, (size_t)step->n_seq * 4));
  }
  // the path
  if (step->n_prompts > 0 && pl.T_p > 0) {
    st = milora_route(ctx, step->layer, w + pl.H, reinterpret_cast<const int32_t*>(w + pl.cu_p),
                      reinterpret_cast<const int32_t*>(w + pl.slot_p), step->n_prompts, pl.T_p, nullptr, nullptr, stream);
    if (st != MILORA_OK) return st;
  }
  bool any_site = false;
  for (int m = 0; m < MILORA_NMOD; ++m) any_site = any_site || step->X_host[m];
  if (step->n_seq > 0 && step->T > 0 && any_site) {
    // Only the rows the method touches cross the link: the host reads the route table back (the one point where
    // the call waits for the stream), and then, module by module, sends the input and base-output rows of the
    // sequences that select this module and fetches the same rows of the output.  Rows of other sequences are
    // never sent: the kernels do not touch them on the device, and their place in Y_host keeps what it held.
    // The link carries both directions at once: the copy of module m's output back to the host runs on a second
    // stream while module m + 1 is being uploaded.
    if (!ctx->copy_ready) {
      MILORA_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
      MILORA_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_done, cudaEventDisableTiming));
      for (int m = 0; m < MILORA_NMOD; ++m)
        MILORA_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_site[m], cudaEventDisableTiming));
      ctx->copy_ready = true;
    }
    int32_t* ws = reinterpret_cast<int32_t*>(w + pl.ws);
    st = milora_group(ctx, step->layer, 1, reinterpret_cast<const int32_t*>(w + pl.cu_s),
                      reinterpret_cast<const int32_t*>(w + pl.slot_s), step->n_seq, step->T, ws, pl.ws_stride, stream);
    if (st != MILORA_OK) return st;
    const int K = top_k_of(ctx), NL = ctx->desc.n_layers;
    try {
      ctx->h_route_copy.resize((size_t)ctx->desc.max_requests * NL * K);
    } catch (...) {
      return MILORA_E_CAPACITY;
    }
    MILORA_CUDA(ctx, cudaMemcpyAsync(ctx->h_route_copy.data(), ctx->d_route, ctx->h_route_copy.size() * sizeof(int32_t),
                                     cudaMemcpyDeviceToHost, s));
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    milora_groups g{ws, step->n_seq, step->T};
    // row ranges of module m: runs of adjacent sequences that select it
    std::vector<std::pair<int, int>> runs;
    for (int m = 0; m < MILORA_NMOD; ++m) {
      if (!step->X_host[m]) continue;
      int d1, d2;
      module_dims(ctx->desc, m, &d1, &d2);
      runs.clear();
      for (int i = 0; i < step->n_seq; ++i) {
        const int slot = step->seq_slot_host[i];
        const int lo = step->cu_seq_host[i], hi = step->cu_seq_host[i + 1];
        if (slot < 0 || slot >= ctx->desc.max_requests || lo < 0 || hi <= lo || hi > step->T) continue;
        bool sel = false;
        for (int j = 0; j < K; ++j) sel = sel || ctx->h_route_copy[((size_t)slot * NL + step->layer) * K + j] == m;
        if (!sel) continue;
        if (!runs.empty() && runs.back().second == lo) runs.back().second = hi;
        else runs.emplace_back(lo, hi);
      }
      if (runs.empty()) continue;
      const char* Xh = static_cast<const char*>(step->X_host[m]);
      char* Yh = static_cast<char*>(step->Y_host[m]);
      for (const auto& r : runs) {
        const size_t rows = (size_t)(r.second - r.first);
        MILORA_CUDA(ctx, cudaMemcpyAsync(w + pl.X[m] + (size_t)r.first * d1 * e, Xh + (size_t)r.first * d1 * e, rows * d1 * e,
                                         cudaMemcpyHostToDevice, s));
        MILORA_CUDA(ctx, cudaMemcpyAsync(w + pl.Y[m] + (size_t)r.first * d2 * e, Yh + (size_t)r.first * d2 * e, rows * d2 * e,
                                         cudaMemcpyHostToDevice, s));
      }
      st = milora_apply_prefill(ctx, step->layer, m, w + pl.X[m], w + pl.Y[m], &g, stream);
      if (st != MILORA_OK) return st;
      st = milora_apply_decode(ctx, step->layer, m, w + pl.X[m], w + pl.Y[m], &g, stream);
      if (st != MILORA_OK) return st;
      MILORA_CUDA(ctx, cudaEventRecord(ctx->ev_site[m], s));
      MILORA_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_site[m], 0));
      for (const auto& r : runs) {
        const size_t rows = (size_t)(r.second - r.first);
        MILORA_CUDA(ctx, cudaMemcpyAsync(Yh + (size_t)r.first * d2 * e, w + pl.Y[m] + (size_t)r.first * d2 * e, rows * d2 * e,
                                         cudaMemcpyDeviceToHost, ctx->copy_stream));
      }
    }
    // the caller's stream is done only when every output has arrived (and the workspace may be reused)
    MILORA_CUDA(ctx, cudaEventRecord(ctx->ev_done, ctx->copy_stream));
    MILORA_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_done, 0));
  }
  return MILORA_OK;
}

milora_status milora_poll_error(milora_ctx* ctx, int* device_flag_out, void* stream) {
  if (!ctx || !device_flag_out) return MILORA_E_ARG;
  cudaStream_t s = as_stream(stream);
  int32_t flag = 0;
  MILORA_CUDA(ctx, cudaMemcpyAsync(&flag, ctx->d_err, sizeof(flag), cudaMemcpyDeviceToHost, s));
  MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  if (flag & ERR_WAIT_TIMEOUT) {
    // a kernel gave up on a wait: its self-cleaning counters may not be back at zero
    ctx->stream_dirty = true;
    ctx->dsplit_dirty = true;
  }
  if (flag) {
    MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_err, 0, sizeof(int32_t), s));
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
  }
  *device_flag_out = flag;
  return flag ? MILORA_E_DEVICE_INDEX : MILORA_OK;
}

}  // extern "C"
