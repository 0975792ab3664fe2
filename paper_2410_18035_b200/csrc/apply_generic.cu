// Generic LoRA apply (Eq. 1 on the routed module): y[row] += s * (x[row] . A) . B for the rows of a
// work list.  Plain SIMT, fp32 accumulation, works for every dtype, rank and shape the context
// accepts.  It is the fp32 path (tensor-core TF32 would not meet a 1e-4 tolerance) and the fallback
// of the specialised bf16 kernels.
//
// One CTA handles up to R rows that share an adapter: phase 1 computes v = x . A with one warp per
// rank row (lanes stride the d1 columns with 128-bit loads, then a shuffle reduction); phase 2 lets
// every thread own 16-byte column groups of y and accumulate sum_j v[j] * B[j][cols].
// Reduction orders are fixed, so results are reproducible run to run.
#include "milora_internal.h"

namespace milora {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxRank = 256;
constexpr int kDenseRows = 8;   // rows per CTA when walking a dense tile

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
  int32_t* err;
  ApplySites sites;
  const int32_t* ws;
  milora_group_layout_t lay;
  int T;
};

template <typename T, bool DENSE>
__global__ void __launch_bounds__(kThreads) apply_generic_kernel(ApplyArgs a) {
  constexpr int V = Elem<T>::V;
  constexpr int R = DENSE ? kDenseRows : kGatherRows;
  constexpr int kSub = DENSE ? kTileRows / R : 1;   // a dense tile is processed as sub-blocks of R rows
  __shared__ float v_sm[R][kMaxRank];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int job_idx = blockIdx.x / kSub, sub = blockIdx.x % kSub;
  pdl_launch_dependents();
  pdl_wait();
  const int n_jobs = a.ws[a.lay.header + (DENSE ? H_NTILES : H_NGATHER)];
  if (job_idx >= n_jobs || job_idx >= (DENSE ? a.lay.max_tiles : a.lay.max_gather)) return;

  const void *At_v, *B_v;
  int r, module, n_rows, rows[R];
  float scale, gate[R];
  if (DENSE) {
    const TileJob w = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles)[job_idx];
    At_v = w.At; B_v = w.B; r = w.rank; scale = w.scale; module = w.module;
    n_rows = min(R, w.count - sub * R);
#pragma unroll
    for (int t = 0; t < R; ++t) {
      rows[t] = (t < n_rows) ? w.start + sub * R + t : -1;
      gate[t] = 1.f;                      // a tile's weight is already folded into its scale
    }
  } else {
    const GatherJob w = reinterpret_cast<const GatherJob*>(a.ws + a.lay.gather)[job_idx];
    At_v = w.At; B_v = w.B; r = w.rank; scale = w.scale; module = w.module;
    n_rows = min(R, w.count);
#pragma unroll
    for (int t = 0; t < R; ++t) {
      rows[t] = (t < n_rows) ? w.rows[t] : -1;
      gate[t] = (t < kGatherRows) ? w.gate[t < kGatherRows ? t : 0] : 0.f;
    }
  }
  if (n_rows <= 0) return;
  int si = -1;
#pragma unroll
  for (int i = 0; i < kMaxSites; ++i)
    if (i < a.sites.n && a.sites.site[i].module == module) si = i;
  if (si < 0) return;                    // this launch does not cover the job's module
  if (r <= 0 || r > kMaxRank || !At_v || !B_v) {
    if (tid == 0) atomicOr(a.err, ERR_BAD_ITEM);
    return;
  }
#pragma unroll
  for (int t = 0; t < R; ++t) {
    if (rows[t] >= a.T || (t < n_rows && rows[t] < 0)) {
      if (tid == 0) atomicOr(a.err, ERR_BAD_ROW);
      rows[t] = -1;
    }
  }
  const ApplySite& site = a.sites.site[si];
  const int d1 = site.d1, d2 = site.d2;
  const T* X = static_cast<const T*>(site.X);
  T* Y = static_cast<T*>(site.Y);
  const T* At = static_cast<const T*>(At_v);
  const T* B = static_cast<const T*>(B_v);

  // ---- phase 1: v[t][j] = s * sum_c x[row_t][c] * At[j][c] ----
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
        if (rows[t] >= 0) {
          float xv[V];
          Elem<T>::load(X + (size_t)rows[t] * d1 + c, xv);
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
      for (int t = 0; t < R; ++t) v_sm[t][j] = acc[t] * scale * gate[t];
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
      if (rows[t] >= 0) {
        float yv[V];
        Elem<T>::load(Y + (size_t)rows[t] * d2 + c, yv);
#pragma unroll
        for (int i = 0; i < V; ++i) yv[i] += out[t][i];
        Elem<T>::store(Y + (size_t)rows[t] * d2 + c, yv);
      }
    }
  }
}

}  // namespace

milora_status launch_apply_generic(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                   bool dense, cudaStream_t s) {
  (void)layer;   // the job records already carry the adapters of their layer
  ApplyArgs a;
  a.err = ctx->d_err;
  a.sites = sites;
  a.ws = g->ws_dev;
  a.lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  a.T = g->T;
  // one CTA per (job, sub-block) of the largest list this batch can have; the exact count is on the device
  size_t grid = dense ? (size_t)a.lay.max_tiles * (kTileRows / kDenseRows) : (size_t)a.lay.max_gather;
  if (grid < 1) grid = 1;
  if (grid > 0x7fffffffull) return MILORA_E_CAPACITY;
  const bool f32 = ctx->desc.dtype == MILORA_F32;
  const dim3 g3((unsigned)grid), b3(kThreads);
  cudaError_t e;
  if (dense) e = f32 ? launch_pdl(apply_generic_kernel<float, true>, g3, b3, 0, s, a)
                     : launch_pdl(apply_generic_kernel<__nv_bfloat16, true>, g3, b3, 0, s, a);
  else e = f32 ? launch_pdl(apply_generic_kernel<float, false>, g3, b3, 0, s, a)
               : launch_pdl(apply_generic_kernel<__nv_bfloat16, false>, g3, b3, 0, s, a);
  MILORA_CUDA(ctx, e);
  MILORA_CUDA(ctx, cudaGetLastError());
  return MILORA_OK;
}

}  // namespace milora
