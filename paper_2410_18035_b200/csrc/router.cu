// Prompt-aware router (Section 3.3, Eq. 2-3; Appendix C; Eq. 7):
// pooling over the prompt's rows -> activation g -> 7 dot products with W_r -> softmax -> argmax,
// written to the int32 route table.
//
// Two launches.  Pass 1 is bound by reading H (e * n_p * d bytes per prompt): a unit is one 64-row chunk of a
// prompt x one strip of 32 sixteen-byte column groups and belongs to ONE WARP, which streams its rows with
// eight independent 128-bit loads per batch, accumulates in fp32 in row order and writes the partial column
// sums to scratch.  Warps take their first unit by index and later ones from an atomic counter (fetched one
// unit ahead); they never synchronise with each other, so every SM has dozens of independent load chains in
// flight.  Pass 2 (one CTA per prompt) adds the partials in chunk order, applies g, does the 7 dot products,
// softmax and argmax.  No fences, no spin-waits; the result does not depend on scheduling.
#include <cfloat>

#include "milora_internal.h"

// Scratch of milora_route_static: partial column sums and chunk statistics, followed by the scheduling
// word.  It lives in the library image, so every GPU that loads
// the library holds it (16 MiB + 16 KiB) until the process exits, and every call of that entry point
// shares it.
constexpr size_t kStaticPartialFloats = size_t(4) << 20;
constexpr size_t kStaticCounters = 4096;
static __device__ __align__(256) float g_route_static_scratch[kStaticPartialFloats + kStaticCounters];

namespace milora {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsMax = 128;   // rows of a chunk: 64 or 128, chosen per call so that one round of units fills the GPU

template <typename T> struct VecOf;
template <> struct VecOf<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    float4 q = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <> struct VecOf<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

__device__ inline float activate(float h, const RouterEntry& r) {
  switch (r.act) {
    case MILORA_ACT_TANH: return tanhf(h);
    case MILORA_ACT_RELU: return fmaxf(h, 0.f);
    case MILORA_ACT_GELU: return 0.5f * h * (1.f + erff(h * 0.70710678118654752f));
    case MILORA_ACT_RATIONAL: {
      // Eq. 7: sum_j a_j x^j / (1 + |sum_i b_i x^i|), both by Horner's rule.
      float num = 0.f;
      for (int j = r.n_a - 1; j >= 0; --j) num = fmaf(num, h, r.coef[j]);
      float den = 0.f;
      for (int i = r.n_b - 1; i >= 0; --i) den = fmaf(den, h, r.coef[r.n_a + i]);
      den *= h;
      return num / (1.f + fabsf(den));
    }
    default: return h;
  }
}

// Sum over the block in a fixed order: lanes by xor-shuffle, then every thread adds the warp totals in order.
template <int NV, int NW>
__device__ inline void block_sum(float (&v)[NV], float* smem /* [NV][NW] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[i] += __shfl_xor_sync(0xffffffffu, v[i], o);
  }
  __syncthreads();
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NV; ++i) smem[i * NW + warp] = v[i];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += smem[i * NW + w];
    v[i] = s;
  }
}

// L2 policies: H is read once (evict first), the partial sums are read back by pass 2 some tens of microseconds
// later, after 268 MB of H have gone through the 126 MB L2 (evict last; pass 2 reads them as evict first again).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_f4_hint(float* p, float4 v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z),
               "f"(v.w), "l"(pol)
               : "memory");
}
__device__ __forceinline__ float4 ld_f4_hint(const float* p, uint64_t pol) {
  float4 v;
  asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p), "l"(pol));
  return v;
}

// 128-bit streaming load that the compiler keeps in program order with the other loads of a batch.
__device__ __forceinline__ uint4 ldg16_stream(const void* p) {
  uint4 q;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
               : "l"(p));
  return q;
}
__device__ __forceinline__ void unpack16(const uint4& q, float (&v)[4]) {
  v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y); v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
}
__device__ __forceinline__ void unpack16(const uint4& q, float (&v)[8]) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// Column reduction over `nr` rows for the 16-byte column group at `col` (row stride d): sum, max, or sum
// weighted by w[t].  Rows are fetched in batches of kDepth independent 128-bit loads and combined in order.
enum { kRedSum = 0, kRedMax = 1, kRedWeighted = 2 };
constexpr int kDepth = 16;
template <typename T, int MODE>
__device__ __forceinline__ void reduce_rows(const T* col, int d, int nr, const float* w, float (&acc)[VecOf<T>::N]) {
  constexpr int V = VecOf<T>::N;
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = MODE == kRedMax ? -FLT_MAX : 0.f;
  auto consume = [&](const uint4& q, int t) {
    float v[V];
    unpack16(q, v);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      if (MODE == kRedMax) acc[i] = fmaxf(acc[i], v[i]);
      else if (MODE == kRedWeighted) acc[i] = fmaf(w[t], v[i], acc[i]);
      else acc[i] += v[i];
    }
  };
  int t = 0;
  for (; t + kDepth <= nr; t += kDepth) {
    uint4 q[kDepth];
#pragma unroll
    for (int k = 0; k < kDepth; ++k) q[k] = ldg16_stream(col + (size_t)(t + k) * d);
#pragma unroll
    for (int k = 0; k < kDepth; ++k) consume(q[k], t + k);
  }
  for (; t < nr; ++t) consume(ldg16_stream(col + (size_t)t * d), t);
}

struct RouteArgs {
  DeviceTables tab;
  const void* H;
  const int32_t* cu;
  const int32_t* seq_slot;
  float* logits_out;
  float* probs_out;
  float* partial;     // [total_chunks][d]
  float* stats;       // [total_chunks][2]  (self-attention pooler: chunk max, chunk sum of exp)
  int32_t* sched;     // next dynamic unit; zero on entry, put back to zero by pass 2
  int layer, P, d, n_strips, rows;
  int T_total;        // rows of H: every row range read from cu is checked against it
  int max_chunks;     // rows of `partial` / `stats`: no unit beyond them is touched
};

// Row range of prompt p.  cu is a device array the host never sees: a range that is negative, reversed or beyond the
// rows of H is treated as empty and raises ERR_BAD_ROW (both passes take the same decision, so the chunk numbering
// stays consistent), and no chunk beyond the scratch the host sized from T_total is touched.
__device__ __forceinline__ void prompt_rows(const RouteArgs& a, int p, int* lo, int* hi) {
  const int l = a.cu[p], h = a.cu[p + 1];
  if (l < 0 || h < l || h > a.T_total) {
    atomicOr(a.tab.err, ERR_BAD_ROW);
    *lo = 0;
    *hi = 0;
  } else {
    *lo = l;
    *hi = h;
  }
}

// Router entry of prompt p, or nullptr when its slot is closed / its tenant has no router at this layer.
__device__ __forceinline__ const RouterEntry* router_of(const RouteArgs& a, int p, int* slot_out) {
  const int slot = a.seq_slot[p];
  *slot_out = slot;
  if (slot < 0 || slot >= a.tab.max_requests) return nullptr;
  const int tenant = a.tab.slot_tenant[slot];
  if (tenant < 0 || tenant >= a.tab.max_tenants) return nullptr;
  const RouterEntry* r = &a.tab.routers[(size_t)tenant * a.tab.n_layers + a.layer];
  return (r->W != nullptr && r->pool >= 0) ? r : nullptr;
}

// ---- pass 1: partial column reductions -------------------------------------------------------------
// A unit is one 64-row chunk of a prompt x one strip of 32 sixteen-byte column groups, handled by ONE
// WARP; warps walk the units with a fixed stride and never synchronise with each other, so an SM always
// has dozens of independent load chains in flight.  Dynamic shared memory: chunk_start[P+1], pool[P].
template <typename T>
__global__ void __launch_bounds__(kThreads) pool_partial_kernel(RouteArgs a) {
  extern __shared__ int32_t sm_i[];
  int32_t* chunk_start = sm_i;
  int32_t* pool_sm = sm_i + (a.P + 1);
  __shared__ int32_t carry;
  __shared__ int32_t wsum[kWarps];
  __shared__ float u_all[kWarps][kRowsMax];
  const int kRows = a.rows;
  constexpr int V = VecOf<T>::N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = a.d;
  const T* H = static_cast<const T*>(a.H);
  const uint64_t pol_part = l2_policy_evict_last();      // the partial sums stay in L2 for pass 2
  // Pass 2 reads the prompt lengths, slots and router table before its own wait; it may do so only once
  // everything ahead of this kernel has completed, so the trigger comes after the wait here.
  pdl_wait();
  pdl_launch_dependents();

  // per-CTA prefix over prompts: chunks per prompt (from the lengths) and the pooler of each prompt
  if (tid == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < a.P; base += kThreads) {
    const int p = base + tid;
    int chunks = 0;
    if (p < a.P) {
      int row_lo, row_hi;
      prompt_rows(a, p, &row_lo, &row_hi);
      const int n_p = row_hi - row_lo;
      if (n_p > 0) chunks = (n_p + kRows - 1) / kRows;
      int slot;
      const RouterEntry* r = router_of(a, p, &slot);
      pool_sm[p] = r ? r->pool : -1;
    }
    int sc = chunks;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int tc = __shfl_up_sync(0xffffffffu, sc, o);
      if (lane >= o) sc += tc;
    }
    if (lane == 31) wsum[warp] = sc;
    __syncthreads();
    int off = carry;
    for (int w = 0; w < warp; ++w) off += wsum[w];
    if (p < a.P) chunk_start[p] = off + sc - chunks;
    __syncthreads();
    if (tid == kThreads - 1) carry = off + sc;
    __syncthreads();
  }
  if (tid == 0) chunk_start[a.P] = carry;
  __syncthreads();
  const int total_units = chunk_start[a.P] * a.n_strips;
  float* u_sm = u_all[warp];

  const int warps_total = gridDim.x * kWarps;
  int u_next = blockIdx.x * kWarps + warp;
  while (u_next < total_units) {
    const int u = u_next;
    {
      // ask for the following unit now; the answer is only needed when this one is done
      int fetched = 0;
      if (lane == 0) fetched = warps_total + atomicAdd(a.sched, 1);
      u_next = __shfl_sync(0xffffffffu, fetched, 0);
    }
    const int cg = u / a.n_strips, strip = u % a.n_strips;
    int lo = 0, hi = a.P;                       // prompt of this chunk: last p with chunk_start[p] <= cg
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (chunk_start[mid] <= cg) lo = mid; else hi = mid;
    }
    const int p = lo;
    const int pool = pool_sm[p];
    if (pool < 0 || cg >= a.max_chunks) continue;
    const int rc = cg - chunk_start[p];
    int row_lo, row_hi;
    prompt_rows(a, p, &row_lo, &row_hi);
    int r0 = row_lo + rc * kRows;
    int nr = min(kRows, row_hi - r0);
    if (pool == MILORA_POOL_LAST) {             // only the prompt's last row is pooled; its last chunk holds it
      if (rc != chunk_start[p + 1] - chunk_start[p] - 1) continue;
      r0 = row_hi - 1;
      nr = 1;
    }
    float* part = a.partial + (size_t)cg * d;
    if (pool == MILORA_POOL_SELFATTN) {
      // Appendix C needs whole rows: the warp of strip 0 does the chunk alone.  u_t = H[t,:] . w_sa, exp weights
      // relative to the chunk max, then the weighted column sums strip by strip.
      if (strip != 0) continue;
      int slot;
      const RouterEntry* r = router_of(a, p, &slot);
      const T* wsa = static_cast<const T*>(r->Wsa);
      for (int t = 0; t < nr; ++t) {
        const T* row = H + (size_t)(r0 + t) * d;
        float acc = 0.f;
        for (int c = lane * V; c < d; c += 32 * V) {
          float hv[V], wv[V];
          VecOf<T>::load(row + c, hv);
          VecOf<T>::load(wsa + c, wv);
#pragma unroll
          for (int i = 0; i < V; ++i) acc = fmaf(hv[i], wv[i], acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) u_sm[t] = acc;
      }
      __syncwarp();
      float m = -FLT_MAX;
      for (int t = 0; t < nr; ++t) m = fmaxf(m, u_sm[t]);
      __syncwarp();
      for (int t = lane; t < nr; t += 32) u_sm[t] = expf(u_sm[t] - m);
      __syncwarp();
      float l = 0.f;
      for (int t = 0; t < nr; ++t) l += u_sm[t];
      if (lane == 0) {
        a.stats[2 * (size_t)cg] = m;
        a.stats[2 * (size_t)cg + 1] = l;
      }
      for (int c0 = lane * V; c0 < d; c0 += 32 * V) {
        float acc[V];
        reduce_rows<T, kRedWeighted>(H + (size_t)r0 * d + c0, d, nr, u_sm, acc);
#pragma unroll
        for (int i = 0; i < V; i += 4)
          st_f4_hint(part + c0 + i, make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]), pol_part);
      }
      __syncwarp();
      continue;
    }
    const int c0 = (strip * 32 + lane) * V;
    if (c0 < d) {
      float acc[V];
      const T* col = H + (size_t)r0 * d + c0;
      if (pool == MILORA_POOL_MAX) reduce_rows<T, kRedMax>(col, d, nr, u_sm, acc);
      else reduce_rows<T, kRedSum>(col, d, nr, u_sm, acc);
#pragma unroll
      for (int i = 0; i < V; i += 4)
        st_f4_hint(part + c0 + i, make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]), pol_part);
    }
  }
}

// ---- pass 1, bulk-copy form (mean and max pooling) ----------------------------------------------------------
// The same chunks and the same partial sums as above, but H comes in through cp.async.bulk: a unit is one chunk of
// a prompt (kRows rows) x one 2 KB strip of columns; the CTA copies 16 rows of the strip per stage (16 bulk copies of
// 2 KB, one mbarrier) through a ring of three stages, so 96 KB per CTA and 192 KB per SM are on their way at any
// time without a register being held for them (a plain read of this form runs at 6.9-7.1 TB/s on a B200; the
// register-fed loads above at 5.3).  256 threads: lane l of each half owns the 16-byte column group l of the strip,
// the first half adds the even rows of a stage, the second half the odd ones, each in row order; the two halves
// meet when the unit ends (even rows + odd rows), so a chunk's sum does not depend on anything but the prompt.
// Thread 0 issues the copies, one stage for every stage consumed, across unit boundaries; units come from the same
// counter as above, asked for one unit ahead.
constexpr int kBulkStages = 3;
constexpr int kBulkStageRows = 16;
constexpr int kBulkStrip = 2048;                                  // bytes of a row per unit
constexpr int kBulkStageBytes = kBulkStageRows * kBulkStrip;
constexpr int kBulkUnitRing = 4;
struct BulkUnit {
  const char* src;      // first row of the unit, at the strip's first byte
  float* part;          // partial sums of the chunk, at the strip's first column
  int32_t n_rows, strip_bytes, pool, valid;
};

__device__ __forceinline__ uint32_t bulk_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bulk_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

template <typename T>
__global__ void __launch_bounds__(kThreads + 32, 2) pool_bulk_kernel(RouteArgs a) {
  extern __shared__ __align__(128) unsigned char sm_raw[];
  unsigned char* ring = sm_raw;
  int32_t* chunk_start = reinterpret_cast<int32_t*>(sm_raw + kBulkStages * kBulkStageBytes);
  int32_t* pool_sm = chunk_start + (a.P + 1);
  int32_t* row_lo_sm = pool_sm + a.P;          // checked row ranges, so that the copy warp never waits for cu_seqlens
  int32_t* row_hi_sm = row_lo_sm + a.P;
  __shared__ int32_t carry;
  __shared__ int32_t wsum[kWarps];
  __shared__ uint64_t full[kBulkStages], empty[kBulkStages];
  __shared__ BulkUnit unit_q[kBulkUnitRing];
  __shared__ float red[kThreads / 2][8];
  __shared__ volatile int32_t s_failed;          // a worker warp gave up on a wait: all of them leave together
  const int kRows = a.rows;
  constexpr int V = VecOf<T>::N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool worker = tid < kThreads;          // warps 0..7 add rows up, warp 8 issues the copies
  const int d = a.d;
  const size_t row_bytes = (size_t)d * sizeof(T);
  if (tid == 0) {
    for (int i = 0; i < kBulkStages; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bulk_smem_u32(&full[i])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bulk_smem_u32(&empty[i])), "r"(kWarps));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    carry = 0;
    s_failed = 0;
  }
  pdl_wait();
  pdl_launch_dependents();
  __syncthreads();

  // per-CTA prefix over prompts: chunks per prompt (from the checked row ranges)
  for (int base = 0; base < a.P; base += kThreads) {
    const int p = base + tid;
    int chunks = 0;
    if (worker && p < a.P) {
      int row_lo, row_hi;
      prompt_rows(a, p, &row_lo, &row_hi);
      row_lo_sm[p] = row_lo;
      row_hi_sm[p] = row_hi;
      const int n_p = row_hi - row_lo;
      if (n_p > 0) chunks = (n_p + kRows - 1) / kRows;
    }
    int sc = chunks;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int tc = __shfl_up_sync(0xffffffffu, sc, o);
      if (lane >= o) sc += tc;
    }
    if (worker && lane == 31) wsum[warp] = sc;
    __syncthreads();
    int off = carry;
    for (int w = 0; w < warp && w < kWarps; ++w) off += wsum[w];
    if (worker && p < a.P) chunk_start[p] = off + sc - chunks;
    __syncthreads();
    if (tid == kThreads - 1) carry = off + sc;
    __syncthreads();
  }
  if (tid == 0) chunk_start[a.P] = carry;
  __syncthreads();
  const int total_units = chunk_start[a.P] * a.n_strips;

  if (!worker) {
    // ---- copy warp: units from the counter (asked for one unit ahead), one stage of 16 row copies at a time,
    //      one lane per row; a stage is refilled as soon as the eight worker warps have handed it back ----
    const uint64_t pol_h = l2_policy_evict_first();
    int u_next = blockIdx.x, n_queued = 0, g_issued = 0;
    uint32_t fetched = 0;
    bool gave_up = false;
    while (!gave_up) {
      const int u = u_next;
      if (u >= total_units) break;
      if (lane == 0) fetched = (uint32_t)gridDim.x + (uint32_t)atomicAdd(a.sched, 1);
      const int cg = u / a.n_strips, strip = u % a.n_strips;
      int lo = 0, hi = a.P;                       // prompt of this chunk: last p with chunk_start[p] <= cg
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (chunk_start[mid] <= cg) lo = mid; else hi = mid;
      }
      const int p = lo;
      const int r0 = row_lo_sm[p] + (cg - chunk_start[p]) * kRows;
      const int nr = min(kRows, row_hi_sm[p] - r0);
      const int sb = (int)min((size_t)kBulkStrip, row_bytes - (size_t)strip * kBulkStrip);
      if (cg < a.max_chunks && nr > 0 && sb > 0) {
        BulkUnit un;
        un.src = static_cast<const char*>(a.H) + (size_t)r0 * row_bytes + (size_t)strip * kBulkStrip;
        un.part = a.partial + (size_t)cg * d + (size_t)strip * (kBulkStrip / sizeof(T));
        un.n_rows = nr; un.strip_bytes = sb; un.pool = p; un.valid = 1;      // pool: the prompt, for now
        if (lane == 0) unit_q[n_queued % kBulkUnitRing] = un;
        ++n_queued;
        const int n_stages = (nr + kBulkStageRows - 1) / kBulkStageRows;
        for (int j = 0; j < n_stages && !gave_up; ++j, ++g_issued) {
          const int st = g_issued % kBulkStages;
          if (g_issued >= kBulkStages) {
            const uint32_t parity = (uint32_t)(g_issued / kBulkStages - 1) & 1u;
            bool freed = false;
            for (uint32_t spin = 0; spin < (4u << 20); ++spin)
              if (bulk_try_wait(bulk_smem_u32(&empty[st]), parity)) { freed = true; break; }
            if (!freed) { gave_up = true; break; }
          }
          const uint32_t bar = bulk_smem_u32(&full[st]);
          const int r_first = j * kBulkStageRows, rows = min(kBulkStageRows, nr - r_first);
          if (lane == 0)
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(rows * sb)) : "memory");
          __syncwarp();
          if (lane < rows)
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                    bulk_smem_u32(ring + st * kBulkStageBytes + lane * kBulkStrip)),
                "l"(un.src + (size_t)(r_first + lane) * row_bytes), "r"((uint32_t)sb), "r"(bar), "l"(pol_h)
                : "memory");
        }
      }
      u_next = (int)__shfl_sync(0xffffffffu, fetched, 0);
    }
    // the end marker travels like a stage: its record, then an arrive on the next stage's barrier
    if (!gave_up) {
      const int st = g_issued % kBulkStages;
      bool freed = g_issued < kBulkStages;
      if (!freed) {
        const uint32_t parity = (uint32_t)(g_issued / kBulkStages - 1) & 1u;
        for (uint32_t spin = 0; spin < (4u << 20); ++spin)
          if (bulk_try_wait(bulk_smem_u32(&empty[st]), parity)) { freed = true; break; }
      }
      if (freed && lane == 0) {
        unit_q[n_queued % kBulkUnitRing].valid = 0;
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bulk_smem_u32(&full[st])) : "memory");
      }
      gave_up = !freed;
    }
    if (gave_up && lane == 0) atomicOr(a.tab.err, ERR_WAIT_TIMEOUT);
    return;
  }

  // ---- worker warps ----
  // The pooler of each prompt sits behind a chain of look-ups (slot, tenant, router entry); it is only needed when
  // rows are added up, so the chain runs while the first copies are on their way.  A prompt without a router has
  // its rows copied for nothing; its units are dropped below.
  for (int p = tid; p < a.P; p += kThreads) {
    int slot;
    const RouterEntry* r = router_of(a, p, &slot);
    pool_sm[p] = r ? r->pool : -1;
  }
  asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
  const int half = tid >> 7, l = tid & 127;
  const uint64_t pol_part = l2_policy_evict_last();
  int g_done = 0;
  auto wait_full = [&](int n) {          // bounded wait for stage number n; a warp that gives up tells the others
    const uint32_t bar = bulk_smem_u32(&full[n % kBulkStages]), parity = (uint32_t)(n / kBulkStages) & 1u;
    for (uint32_t spin = 0; spin < (4u << 20); ++spin)
      if (bulk_try_wait(bar, parity)) return true;
    s_failed = 1;
    return false;
  };
  for (int k = 0;; ++k) {
    // the unit's record is released by the arrive on its first stage's barrier
    BulkUnit un;
    un.valid = 0;
    un.n_rows = 0;
    bool ok = wait_full(g_done);
    if (ok) un = unit_q[k % kBulkUnitRing];
    if (ok && !un.valid) break;            // the end marker: every worker warp sees it
    const int pool = ok ? pool_sm[un.pool] : -1;
    const bool is_max = pool == MILORA_POOL_MAX;
    const bool col_ok = ok && l * 16 < un.strip_bytes && pool >= 0;
    float acc[V];
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = is_max ? -FLT_MAX : 0.f;
    const int n_stages = ok ? (un.n_rows + kBulkStageRows - 1) / kBulkStageRows : 0;
    for (int j = 0; j < n_stages && ok; ++j, ++g_done) {
      const int st = g_done % kBulkStages;
      if (j > 0) ok = wait_full(g_done);
      if (!ok) break;
      const int rows = min(kBulkStageRows, un.n_rows - j * kBulkStageRows);
      if (col_ok) {
        const unsigned char* base = ring + st * kBulkStageBytes + l * 16;
        if (is_max) {
#pragma unroll 8
          for (int r = half; r < rows; r += 2) {
            float v[V];
            unpack16(*reinterpret_cast<const uint4*>(base + r * kBulkStrip), v);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = fmaxf(acc[i], v[i]);
          }
        } else {
#pragma unroll 8
          for (int r = half; r < rows; r += 2) {
            float v[V];
            unpack16(*reinterpret_cast<const uint4*>(base + r * kBulkStrip), v);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] += v[i];
          }
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bulk_smem_u32(&empty[st])) : "memory");
    }
    // the halves meet: even rows + odd rows.  Every worker warp reaches these two barriers, also one that gave up.
    if (half == 1 && col_ok) {
#pragma unroll
      for (int i = 0; i < V; ++i) red[l][i] = acc[i];
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
    const bool stop = s_failed != 0;
    if (half == 0 && col_ok && !stop) {
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = is_max ? fmaxf(acc[i], red[l][i]) : acc[i] + red[l][i];
      float* dst = un.part + l * V;
#pragma unroll
      for (int i = 0; i < V; i += 4) st_f4_hint(dst + i, make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]), pol_part);
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");      // red is reused by the next unit
    if (stop) break;
  }
  if (s_failed && tid == 0) atomicOr(a.tab.err, ERR_WAIT_TIMEOUT);
}

// ---- pass 2: one CTA per prompt combines the partials in chunk order and routes -----------------------
// 512 threads: at d = 4096 (bf16) every thread owns one 16-byte column group, so the chain a warp has to run
// after pass 1 has finished (fetch the partial sums, eight accurate tanh, 56 multiply-adds) is gone through once.
constexpr int kFinThreads = 512;
constexpr int kFinWarps = kFinThreads / 32;
template <typename T>
__global__ void __launch_bounds__(kFinThreads) route_finalize_kernel(RouteArgs a) {
  constexpr int V = VecOf<T>::N;
  const int kRows = a.rows;
  __shared__ float red[MILORA_NMOD * kFinWarps];
  __shared__ int32_t wsum[kFinWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int p = blockIdx.x, d = a.d;
  // Launched behind pass 1, whose CTAs trigger only after their own wait: lengths, slots and tables are final
  // when this CTA starts, so its look-ups overlap the tail of pass 1.  Only the partial sums need pdl_wait().
  pdl_launch_dependents();
  // first scratch row of this prompt = number of chunks of the prompts before it
  int mine = 0;
  for (int q = tid; q < p; q += kFinThreads) {
    int q_lo, q_hi;
    prompt_rows(a, q, &q_lo, &q_hi);
    const int n_q = q_hi - q_lo;
    if (n_q > 0) mine += (n_q + kRows - 1) / kRows;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
  if (lane == 0) wsum[warp] = mine;
  __syncthreads();
  int chunk0 = 0;
  for (int w = 0; w < kFinWarps; ++w) chunk0 += wsum[w];
  int p_lo, p_hi;
  prompt_rows(a, p, &p_lo, &p_hi);
  const int n_p = p_hi - p_lo;
  int n_chunks = n_p > 0 ? (n_p + kRows - 1) / kRows : 0;
  // chunks beyond the scratch do not exist for pass 1 either: such a prompt stays "not routed"
  if (chunk0 + n_chunks > a.max_chunks) n_chunks = 0;
  int slot;
  const RouterEntry* rp = router_of(a, p, &slot);
  if (!rp || n_chunks == 0) {
    // closed slot, no router for this tenant at this layer, or an empty prompt: the request stays "not routed"
    pdl_wait();
    if (tid == 0) {
      if (slot >= 0 && slot < a.tab.max_requests) {
        for (int j = 0; j < a.tab.top_k; ++j)
          a.tab.route[((size_t)slot * a.tab.n_layers + a.layer) * a.tab.top_k + j] = -1;
      } else {
        atomicOr(a.tab.err, ERR_BAD_SLOT);
      }
      if (p == 0) *a.sched = 0;
    }
    return;
  }
  const RouterEntry& r = *rp;
  const int pool = r.pool;
  const bool sa = pool == MILORA_POOL_SELFATTN;
  if (pool == MILORA_POOL_LAST) { chunk0 += n_chunks - 1; n_chunks = 1; }   // only the chunk with the last row counts
  const float* part0 = a.partial + (size_t)chunk0 * d;
  const float* st0 = a.stats + 2 * (size_t)chunk0;
  pdl_wait();                                   // the partial sums of pass 1
  const uint64_t pol_read = l2_policy_evict_first();
  float gmax = -FLT_MAX, denom = 1.f;
  if (sa) {
    for (int c = 0; c < n_chunks; ++c) gmax = fmaxf(gmax, st0[2 * c]);
    denom = 0.f;
    for (int c = 0; c < n_chunks; ++c) denom += expf(st0[2 * c] - gmax) * st0[2 * c + 1];
  }
  const T* W = static_cast<const T*>(r.W);
  float z[MILORA_NMOD];
#pragma unroll
  for (int j = 0; j < MILORA_NMOD; ++j) z[j] = 0.f;
  for (int c0 = tid * V; c0 < d; c0 += kFinThreads * V) {
    float h[V];
#pragma unroll
    for (int i = 0; i < V; ++i) h[i] = pool == MILORA_POOL_MAX ? -FLT_MAX : 0.f;
    // chunks are fetched eight at a time (all loads of a batch independent) and combined in chunk order
    for (int cbase = 0; cbase < n_chunks; cbase += 8) {
      float4 q[8][V / 4];
      float wgt[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int c = min(cbase + k, n_chunks - 1);
        wgt[k] = sa ? st0[2 * c] : 0.f;
#pragma unroll
        for (int i = 0; i < V / 4; ++i)
          q[k][i] = ld_f4_hint(part0 + (size_t)c * d + c0 + 4 * i, pol_read);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (cbase + k < n_chunks) {
          const float wk = sa ? expf(wgt[k] - gmax) : 1.f;
#pragma unroll
          for (int i = 0; i < V / 4; ++i) {
            const float4 u = q[k][i];
            float* hh = h + 4 * i;
            if (pool == MILORA_POOL_MAX) {
              hh[0] = fmaxf(hh[0], u.x); hh[1] = fmaxf(hh[1], u.y); hh[2] = fmaxf(hh[2], u.z); hh[3] = fmaxf(hh[3], u.w);
            } else if (sa) {
              hh[0] = fmaf(wk, u.x, hh[0]); hh[1] = fmaf(wk, u.y, hh[1]); hh[2] = fmaf(wk, u.z, hh[2]); hh[3] = fmaf(wk, u.w, hh[3]);
            } else {
              hh[0] += u.x; hh[1] += u.y; hh[2] += u.z; hh[3] += u.w;
            }
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < V; ++i) {
      float hv = h[i];
      if (pool == MILORA_POOL_MEAN) hv = hv / (float)n_p;
      else if (sa) hv = hv / denom;
      h[i] = activate(hv, r);
    }
#pragma unroll
    for (int j = 0; j < MILORA_NMOD; ++j) {
      float wv[V];
      VecOf<T>::load(W + (size_t)j * d + c0, wv);
#pragma unroll
      for (int i = 0; i < V; ++i) z[j] = fmaf(h[i], wv[i], z[j]);
    }
  }
  block_sum<MILORA_NMOD, kFinWarps>(z, red);
  if (tid == 0) {
    float zmax = -FLT_MAX;
#pragma unroll
    for (int j = 0; j < MILORA_NMOD; ++j) {
      z[j] += r.bias[j];
      zmax = fmaxf(zmax, z[j]);
    }
    float e[MILORA_NMOD], sum = 0.f;
#pragma unroll
    for (int j = 0; j < MILORA_NMOD; ++j) { e[j] = expf(z[j] - zmax); sum += e[j]; }
    // Eq. 3, Top-k: the k largest in descending order; the comparison is strict, so ties keep the lower index
    const size_t cell = ((size_t)slot * a.tab.n_layers + a.layer) * a.tab.top_k;
    unsigned taken = 0;
    for (int q = 0; q < a.tab.top_k; ++q) {
      int best = -1;
      float bz = 0.f, be = 0.f;
#pragma unroll
      for (int j = 0; j < MILORA_NMOD; ++j) {
        if (!((taken >> j) & 1u) && (best < 0 || z[j] > bz)) { best = j; bz = z[j]; be = e[j]; }
      }
      taken |= 1u << best;
      a.tab.route[cell + q] = best;
      a.tab.gate[cell + q] = be / sum;
    }
    if (p == 0) *a.sched = 0;       // pass 1 of the next call starts its unit queue from zero
    if (a.logits_out) {
#pragma unroll
      for (int j = 0; j < MILORA_NMOD; ++j) a.logits_out[(size_t)p * MILORA_NMOD + j] = z[j];
    }
    if (a.probs_out) {
#pragma unroll
      for (int j = 0; j < MILORA_NMOD; ++j) a.probs_out[(size_t)p * MILORA_NMOD + j] = e[j] / sum;
    }
  }
}

// ---- registration-time repacking -----------------------------------------------------------
// out[j][i] = in[i][j] for in of shape rows x cols (tiled through shared memory).
template <typename T>
__global__ void transpose_kernel(const T* __restrict__ in, T* __restrict__ out, int rows, int cols) {
  __shared__ T tile[32][33];
  int c = blockIdx.x * 32 + threadIdx.x;
  for (int k = threadIdx.y; k < 32; k += blockDim.y) {
    int rr = blockIdx.y * 32 + k;
    if (rr < rows && c < cols) tile[k][threadIdx.x] = in[(size_t)rr * cols + c];
  }
  __syncthreads();
  int orow0 = blockIdx.x * 32, ocol = blockIdx.y * 32 + threadIdx.x;
  for (int k = threadIdx.y; k < 32; k += blockDim.y) {
    int orow = orow0 + k;
    if (orow < cols && ocol < rows) out[(size_t)orow * rows + ocol] = tile[threadIdx.x][k];
  }
}

template <typename T>
milora_status transpose(milora_ctx* ctx, const void* in, void* out, int rows, int cols, cudaStream_t s) {
  dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
  transpose_kernel<T><<<grid, block, 0, s>>>(static_cast<const T*>(in), static_cast<T*>(out), rows, cols);
  MILORA_CUDA(ctx, cudaGetLastError());
  return MILORA_OK;
}

struct RoutePlan {
  int n_strips, rows;
  size_t max_chunks, scratch_floats, max_units;
  int T_total;
  bool bulk;      // pass 1 through bulk copies (every registered router pools by mean or max)
};

RoutePlan plan_route(const milora_ctx* ctx, int P, int T_total) {
  RoutePlan pl;
  const int d = ctx->desc.d_model;
  const int V = ctx->desc.dtype == MILORA_F32 ? 4 : 8;
  pl.n_strips = (d + 32 * V - 1) / (32 * V);
  // 128-row chunks when that still gives every resident warp about one unit (a warp then streams 64 KB without
  // coming back to the queue); 64-row chunks for smaller batches, which need the parallelism
  const size_t warp_slots = (size_t)ctx->sm_count * 5 * kWarps;
  const size_t units128 = ((size_t)T_total / 128 + P) * pl.n_strips;
  pl.rows = units128 * 10 >= warp_slots * 6 ? 128 : 64;
  // Last-token and self-attention pooling need whole rows or a single row: they keep the register-fed kernel.
  pl.bulk = ctx->n_routers_whole_row == 0;
  if (pl.bulk) {
    // 2 KB strips of 64-row chunks: at config 2 that is 2048 units for 296 CTAs, seven rounds with a thin last one
    pl.n_strips = (int)(((size_t)d * ctx->elem + kBulkStrip - 1) / kBulkStrip);
    pl.rows = 64;
  }
  const int kRows = pl.rows;
  pl.max_chunks = (size_t)T_total / kRows + P;
  pl.scratch_floats = pl.max_chunks * d + 2 * pl.max_chunks;
  pl.max_units = pl.max_chunks * pl.n_strips;
  pl.T_total = T_total;
  return pl;
}

// `scratch` holds plan.scratch_floats floats; `sched` is one zeroed int32.
milora_status run_route(milora_ctx* ctx, const RoutePlan& pl, int layer, const void* H, const int32_t* cu,
                        const int32_t* seq_slot, int P, float* logits_out, float* probs_out, float* scratch, int32_t* sched,
                        cudaStream_t s) {
  RouteArgs a;
  a.tab = device_tables(ctx);
  a.H = H; a.cu = cu; a.seq_slot = seq_slot;
  a.logits_out = logits_out; a.probs_out = probs_out;
  a.partial = scratch;
  a.stats = scratch + pl.max_chunks * ctx->desc.d_model;
  a.sched = sched;
  a.layer = layer; a.P = P; a.d = ctx->desc.d_model; a.n_strips = pl.n_strips; a.rows = pl.rows;
  a.T_total = pl.T_total; a.max_chunks = (int)pl.max_chunks;
  RoutePlan plan = pl;
  if (plan.bulk && (reinterpret_cast<uintptr_t>(H) & 15)) {
    // bulk copies want 16-byte aligned rows; the scratch is large enough for either plan (64-row chunks need most)
    plan.bulk = false;
    const int V = ctx->desc.dtype == MILORA_F32 ? 4 : 8;
    a.n_strips = plan.n_strips = (ctx->desc.d_model + 32 * V - 1) / (32 * V);
    plan.max_units = plan.max_chunks * plan.n_strips;
  }
  const size_t smem = (size_t)(2 * P + 1) * sizeof(int32_t);
  const size_t bulk_tables = (size_t)(4 * P + 1) * sizeof(int32_t);
  const bool f32 = ctx->desc.dtype == MILORA_F32;
  // pass 1: one wave of resident CTAs (a warp's first unit is assigned by index, so every CTA must start at once)
  int per_sm = 0;
  if (f32) MILORA_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pool_partial_kernel<float>, kThreads, smem));
  else MILORA_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pool_partial_kernel<__nv_bfloat16>, kThreads, smem));
  if (per_sm < 1) per_sm = 1;
  int grid = (int)std::min<size_t>((plan.max_units + kWarps - 1) / kWarps, (size_t)ctx->sm_count * per_sm);
  if (grid < 1) grid = 1;
  if (plan.bulk) {
    const size_t bsmem = (size_t)kBulkStages * kBulkStageBytes + bulk_tables;
    if (!ctx->route_bulk_attr_set) {
      MILORA_CUDA(ctx, cudaFuncSetAttribute(pool_bulk_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 140 * 1024));
      MILORA_CUDA(ctx, cudaFuncSetAttribute(pool_bulk_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 140 * 1024));
      ctx->route_bulk_attr_set = true;
    }
    const int bgrid = (int)std::max<size_t>(1, std::min<size_t>((size_t)ctx->sm_count * 2, plan.max_units));
    if (f32) MILORA_CUDA(ctx, launch_pdl(pool_bulk_kernel<float>, dim3(bgrid), dim3(kThreads + 32), bsmem, s, a));
    else MILORA_CUDA(ctx, launch_pdl(pool_bulk_kernel<__nv_bfloat16>, dim3(bgrid), dim3(kThreads + 32), bsmem, s, a));
  } else if (f32) MILORA_CUDA(ctx, launch_pdl(pool_partial_kernel<float>, dim3(grid), dim3(kThreads), smem, s, a));
  else MILORA_CUDA(ctx, launch_pdl(pool_partial_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), smem, s, a));
  // pass 2: one CTA per prompt
  if (f32) MILORA_CUDA(ctx, launch_pdl(route_finalize_kernel<float>, dim3(P), dim3(kFinThreads), 0, s, a));
  else MILORA_CUDA(ctx, launch_pdl(route_finalize_kernel<__nv_bfloat16>, dim3(P), dim3(kFinThreads), 0, s, a));
  return MILORA_OK;
}

}  // namespace

milora_status launch_repack_adapter(milora_ctx* ctx, const void* A, const void* B, void* At, void* Bout, int d1, int d2,
                                    int rank, cudaStream_t s) {
  milora_status st = ctx->desc.dtype == MILORA_F32 ? transpose<float>(ctx, A, At, d1, rank, s)
                                                   : transpose<__nv_bfloat16>(ctx, A, At, d1, rank, s);
  if (st != MILORA_OK) return st;
  MILORA_CUDA(ctx, cudaMemcpyAsync(Bout, B, (size_t)rank * d2 * ctx->elem, cudaMemcpyDeviceToDevice, s));
  return MILORA_OK;
}

milora_status launch_repack_router(milora_ctx* ctx, const void* Wr, void* Wt, int d, cudaStream_t s) {
  return ctx->desc.dtype == MILORA_F32 ? transpose<float>(ctx, Wr, Wt, d, MILORA_NMOD, s)
                                       : transpose<__nv_bfloat16>(ctx, Wr, Wt, d, MILORA_NMOD, s);
}

milora_status launch_route(milora_ctx* ctx, int layer, const void* H, const int32_t* cu, const int32_t* seq_slot, int P,
                           int T_total, float* logits_out, float* probs_out, cudaStream_t s) {
  const RoutePlan pl = plan_route(ctx, P, T_total);
  if (pl.scratch_floats > ctx->scratch_floats) {
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    if (ctx->d_scratch) MILORA_CUDA(ctx, cudaFree(ctx->d_scratch));
    ctx->d_scratch = nullptr;
    ctx->scratch_floats = 0;
    MILORA_CUDA(ctx, cudaMalloc(&ctx->d_scratch, pl.scratch_floats * sizeof(float)));
    ctx->scratch_floats = pl.scratch_floats;
  }
  if (ctx->n_counters < 1) {
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    if (ctx->d_counters) MILORA_CUDA(ctx, cudaFree(ctx->d_counters));
    ctx->d_counters = nullptr;
    ctx->n_counters = 0;
    size_t n = 64;
    MILORA_CUDA(ctx, cudaMalloc(&ctx->d_counters, n * sizeof(int32_t)));
    MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_counters, 0, n * sizeof(int32_t), s));
    ctx->n_counters = n;
  }
  return run_route(ctx, pl, layer, H, cu, seq_slot, P, logits_out, probs_out, ctx->d_scratch, ctx->d_counters, s);
}

// Same kernel as launch_route, but the scratch is the file-scope device array above, so that nothing is
// allocated.  In host code the array's name is only a handle: its device address is looked up once per
// device with cudaGetSymbolAddress (with that device current) and cached.
milora_status launch_route_static(milora_ctx* ctx, int layer, const void* H, const int32_t* cu, const int32_t* seq_slot,
                                  int P, int T_total, float* logits_out, float* probs_out, cudaStream_t s) {
  constexpr int kMaxDevices = 64;
  static float* scratch_of_device[kMaxDevices] = {nullptr};
  const RoutePlan pl = plan_route(ctx, P, T_total);
  // the scheduling word sits right behind the partial area.  The documented limit is the need with 64-row
  // chunks, whatever chunk size this call ends up using.
  const size_t documented_need = ((size_t)T_total / 64 + P) * ((size_t)ctx->desc.d_model + 2);
  if (documented_need > kStaticPartialFloats || pl.scratch_floats > kStaticPartialFloats || (size_t)P > kStaticCounters)
    return MILORA_E_CAPACITY;
  int dev = -1;
  MILORA_CUDA(ctx, cudaGetDevice(&dev));
  if (dev != ctx->device) return MILORA_E_STATE;     // the context's device must be current
  if (dev < 0 || dev >= kMaxDevices) return MILORA_E_CAPACITY;
  if (!scratch_of_device[dev]) {
    float* ptr = nullptr;
    MILORA_CUDA(ctx, cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_route_static_scratch));
    scratch_of_device[dev] = ptr;
  }
  float* scratch = scratch_of_device[dev];
  int32_t* sched = reinterpret_cast<int32_t*>(scratch + kStaticPartialFloats);
  // The array keeps whatever the previous call left; only the scheduling word has to start at zero.
  MILORA_CUDA(ctx, cudaMemsetAsync(sched, 0, sizeof(int32_t), s));
  return run_route(ctx, pl, layer, H, cu, seq_slot, P, logits_out, probs_out, scratch, sched, s);
}

}  // namespace milora
