// Generic LoRA apply (Eq. 1 on the routed module): y[row] += s * (x[row] . A) . B for the rows of a
// work list.  Plain SIMT, fp32 accumulation, works for every dtype, rank and shape the context
// accepts.  It is the fp32 path (tensor-core TF32 would not meet a 1e-4 tolerance) and the fallback
// of the specialised bf16 kernels.
//
// One CTA handles up to kGatherRows rows that share an adapter: phase 1 computes v = x . A with one
// warp per rank row (lanes stride the d1 columns with 128-bit loads, then a shuffle reduction);
// phase 2 lets every thread own 16-byte column groups of y and accumulate sum_j v[j] * B[j][cols].
// Reduction orders are fixed, so results are reproducible run to run.
#include "milora_internal.h"

namespace milora {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxRank = 256;

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int V = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
  __device__ static void store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int V = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

struct ApplyArgs {
  DeviceTables tab;
  ApplySites sites;
  const int32_t* ws;
  milora_group_layout_t lay;
  int layer, T;
};

template <typename T, bool DENSE>
__global__ void __launch_bounds__(kThreads) apply_generic_kernel(ApplyArgs a) {
  constexpr int V = Elem<T>::V;
  constexpr int R = kGatherRows;
  __shared__ float v_sm[R][kMaxRank];
  __shared__ int32_t rows_sm[R];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* ws = a.ws;
  const int32_t* mod_off = ws + (DENSE ? a.lay.mod_tile_offset : a.lay.mod_gather_offset);
  const WorkItem* items = reinterpret_cast<const WorkItem*>(ws + (DENSE ? a.lay.tiles : a.lay.gather));
  const int32_t* gather_rows = ws + a.lay.gather_rows;
  const int32_t* seg_key = ws + a.lay.seg_key;
  constexpr int kSub = DENSE ? kTileRows / R : 1;   // a dense tile is processed as sub-blocks of R rows

  // units of this launch: the work items of every site's module, back to back
  int site_begin[kMaxSites + 1];
  site_begin[0] = 0;
#pragma unroll
  for (int i = 0; i < kMaxSites; ++i) {
    int n = 0;
    if (i < a.sites.n) {
      int m = a.sites.site[i].module;
      n = (mod_off[m + 1] - mod_off[m]) * kSub;
    }
    site_begin[i + 1] = site_begin[i] + n;
  }
  const int total = site_begin[kMaxSites];

  for (int u = blockIdx.x; u < total; u += gridDim.x) {
    int si = 0;
#pragma unroll
    for (int i = 1; i < kMaxSites; ++i) si += (u >= site_begin[i]) ? 1 : 0;
    const ApplySite& site = a.sites.site[si];
    const int local = u - site_begin[si];
    const int item_idx = mod_off[site.module] + local / kSub;
    const int sub = local % kSub;
    if (item_idx < 0 || item_idx >= (DENSE ? a.lay.max_tiles : a.lay.max_gather)) {
      if (tid == 0) atomicOr(a.tab.err, ERR_BAD_ITEM);
      continue;
    }
    const WorkItem w = items[item_idx];
    int n_rows = DENSE ? min(R, w.count - sub * R) : min(R, w.count);
    if (n_rows <= 0) continue;   // uniform across the CTA
    __syncthreads();             // v_sm / rows_sm of the previous unit are no longer read
    if (tid < R) {
      int row = -1;
      if (tid < n_rows) {
        row = DENSE ? w.start + sub * R + tid : gather_rows[w.start + tid];
        if (row < 0 || row >= a.T) { row = -1; atomicOr(a.tab.err, ERR_BAD_ROW); }
      }
      rows_sm[tid] = row;
    }
    const int key = seg_key[w.seg];
    const int tenant = key % a.tab.max_tenants;
    const AdapterEntry ent = a.tab.adapters[adapter_index(tenant, a.layer, site.module, a.tab.n_layers)];
    const int r = ent.rank;
    if (r <= 0 || r > kMaxRank || key / a.tab.max_tenants != site.module) {
      if (tid == 0) atomicOr(a.tab.err, ERR_BAD_ITEM);
      continue;
    }
    __syncthreads();
    const int d1 = site.d1, d2 = site.d2;
    const T* X = static_cast<const T*>(site.X);
    T* Y = static_cast<T*>(site.Y);
    const T* At = static_cast<const T*>(ent.At);
    const T* B = static_cast<const T*>(ent.B);

    // ---- phase 1: v[t][j] = sum_c x[row_t][c] * At[j][c] ----
    for (int j = warp; j < r; j += kWarps) {
      float acc[R];
#pragma unroll
      for (int t = 0; t < R; ++t) acc[t] = 0.f;
      const T* arow = At + (size_t)j * d1;
      for (int c = lane * V; c < d1; c += 32 * V) {
        float av[V];
        Elem<T>::load(arow + c, av);
#pragma unroll
        for (int t = 0; t < R; ++t) {
          int row = rows_sm[t];
          if (row >= 0) {
            float xv[V];
            Elem<T>::load(X + (size_t)row * d1 + c, xv);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[t] = fmaf(xv[i], av[i], acc[t]);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < R; ++t) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], o);
      }
      if (lane == 0) {
#pragma unroll
        for (int t = 0; t < R; ++t) v_sm[t][j] = acc[t] * ent.scale;
      }
    }
    __syncthreads();

    // ---- phase 2: y[row_t][c] += sum_j v[t][j] * B[j][c] ----
    for (int c = tid * V; c < d2; c += kThreads * V) {
      float out[R][V];
#pragma unroll
      for (int t = 0; t < R; ++t) {
#pragma unroll
        for (int i = 0; i < V; ++i) out[t][i] = 0.f;
      }
      for (int j = 0; j < r; ++j) {
        float bv[V];
        Elem<T>::load(B + (size_t)j * d2 + c, bv);
#pragma unroll
        for (int t = 0; t < R; ++t) {
          float vj = v_sm[t][j];
#pragma unroll
          for (int i = 0; i < V; ++i) out[t][i] = fmaf(vj, bv[i], out[t][i]);
        }
      }
#pragma unroll
      for (int t = 0; t < R; ++t) {
        int row = rows_sm[t];
        if (row >= 0) {
          float yv[V];
          Elem<T>::load(Y + (size_t)row * d2 + c, yv);
#pragma unroll
          for (int i = 0; i < V; ++i) yv[i] += out[t][i];
          Elem<T>::store(Y + (size_t)row * d2 + c, yv);
        }
      }
    }
  }
}

}  // namespace

milora_status launch_apply_generic(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                   bool dense, cudaStream_t s) {
  ApplyArgs a;
  a.tab = device_tables(ctx);
  a.sites = sites;
  a.ws = g->ws_dev;
  a.lay = group_layout(g->n_seq, g->T);
  a.layer = layer;
  a.T = g->T;
  // upper bound of the units this launch can have (the exact count lives on the device)
  size_t max_units = dense ? (size_t)a.lay.max_tiles * (kTileRows / kGatherRows) : (size_t)a.lay.max_gather;
  int grid = (int)std::min<size_t>(max_units, (size_t)ctx->sm_count * 8);
  if (grid < 1) grid = 1;
  const bool f32 = ctx->desc.dtype == MILORA_F32;
  if (dense) {
    if (f32) apply_generic_kernel<float, true><<<grid, kThreads, 0, s>>>(a);
    else apply_generic_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, s>>>(a);
  } else {
    if (f32) apply_generic_kernel<float, false><<<grid, kThreads, 0, s>>>(a);
    else apply_generic_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, s>>>(a);
  }
  MILORA_CUDA(ctx, cudaGetLastError());
  return MILORA_OK;
}

}  // namespace milora
