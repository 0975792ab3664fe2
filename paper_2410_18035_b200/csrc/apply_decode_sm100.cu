// Decode path of Eq. 1 for bf16 on sm_100a: y[row] += s * (x[row] . A) . B for the gathered rows of the
// decode work list (rows of short sequences, at most kGatherRows per job, all sharing one adapter).
//
// The step is bound by streaming each active adapter once from HBM (r * (d1 + d2) * 2 bytes), so the
// design is about getting every byte requested at once:
//   * one thread-block cluster of kC CTAs per job; CTA c owns a 1/kC slice of the d1 columns (shrink)
//     and a 1/kC slice of the d2 columns (expand);
//   * at start every thread asks for its lines of the A^T and x slices with L2 prefetches, one warp issues
//     bulk copies (cp.async.bulk, completion on an mbarrier) for the CTA's slice of B, and every thread loads
//     its 16-byte pieces of y into registers: the whole job is in flight before anything is consumed;
//   * the A^T slice is then consumed from global memory with 128-bit loads, four per thread per batch
//     (it is read once, so staging it in shared memory would only cost occupancy); later batches hit L2;
//   * each CTA reduces its d1 slice to partial sums v_c[row][j]; the partials go to every CTA of the cluster
//     through distributed shared memory with st.async, which counts their arrival on the receiver's
//     mbarrier (no cluster-wide barrier), and are added in CTA order (deterministic); then each CTA
//     finishes its d2 slice and writes y with 128-bit stores.
// No scratch in global memory, no atomics.  Every wait is bounded; a timeout raises ERR_WAIT_TIMEOUT.
#include "milora_internal.h"

namespace milora {
namespace {

constexpr int kC = 8;              // CTAs per cluster (portable maximum)
constexpr int kThreads = 256;
constexpr int kR = kGatherRows;
constexpr int kSegs = 16;          // threads that share one rank row in the shrink
constexpr int kRowsPerPass = kThreads / kSegs;
constexpr uint32_t kSpinLimit = 4u << 20;
constexpr int kYIter = 4;          // 16-byte pieces of y a thread may own (kR * per2max <= kYIter * kThreads)
constexpr int kUnroll = 4;         // A^T loads a thread keeps in flight

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// Bounded wait; returns false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// "This CTA is running and its barriers are initialised" (made visible by fence.mbarrier_init before it):
// nothing else has to be released, so the arrive is relaxed.
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// One fp32 value into the same shared-memory location of CTA `peer` of the cluster; its arrival is counted
// (4 bytes) on that CTA's mbarrier, so the receiver needs no cluster-wide barrier to know the data is there.
__device__ __forceinline__ void st_async_f32(uint32_t local_addr, uint32_t local_bar, uint32_t peer, float v) {
  uint32_t remote, remote_bar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(peer));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote_bar) : "r"(local_bar), "r"(peer));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(remote),
               "r"(__float_as_uint(v)), "r"(remote_bar)
               : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 q;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
               : "l"(p));
  return q;
}

__device__ __forceinline__ void unpack8(const uint4& q, float (&v)[8]) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&v)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

struct DecodeArgs {
  int32_t* err;
  ApplySites sites;
  const int32_t* ws;
  milora_group_layout_t lay;
  int T;
  int rmax;        // rank rows reserved in shared memory
  int per2max;     // 16-byte column groups reserved per row of the B staging
  int resident;    // clusters the GPU holds at once: job i + resident is the one that follows job i on its SMs
};

// L2 prefetch of `nrows` row slices of `slice_bytes` bytes each (rows `pitch` bytes apart), spread over the CTA.
__device__ __forceinline__ void prefetch_rows(const char* base, size_t pitch, int nrows, size_t slice_bytes, int tid) {
  if (slice_bytes == 0) return;
  const int n_lines = (int)((slice_bytes + 127) / 128) + 1;
  for (int idx = tid; idx < nrows * n_lines; idx += kThreads) {
    const int j = idx / n_lines, l = idx % n_lines;
    prefetch_l2(base + (size_t)j * pitch + min((size_t)l * 128, slice_bytes - 16));
  }
}

// Shared memory (dynamic): [0,32) mbarriers | record of the following job x 2 | part[2][kC][kR][rmax] f32 |
//                          mine[kR][rmax] f32 | v[kR][rmax] f32 | B[rmax][per2max] uint4
// STAGE_B: the CTA's B slice is staged in shared memory by bulk copies.  When rank x d2 is so large that this
// would cost occupancy, it is prefetched into L2 and read from global memory instead (STAGE_B = false).
// LOOP = false: one cluster per slot of the job list (a decode batch: the list is about as long as the number
// of jobs).  LOOP = true: as many clusters as the GPU holds, each walking the list with that stride - for mixed
// batches, whose list is sized for the worst case (every row short) while most rows are prompt rows, so that
// launching one cluster per slot would cost more than the jobs themselves.  Clusters take the list from its
// end: it is ordered by module, and the modules with the most bytes (gate, up, down) come last, so the longest
// jobs start first and the short ones fill the tail.
// In the loop the partial-sum buffers and their barriers alternate by job parity: a peer can be at most one job
// ahead (it needs this CTA's partial sums of job i + 1 to get past it), so the stores for job i + 2 never meet a
// buffer that is still being read.
template <bool STAGE_B, bool LOOP>
__global__ void __cluster_dims__(kC, 1, 1) __launch_bounds__(kThreads, 4) decode_bf16_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t crank = cluster_ctarank();
  const int cluster_id = blockIdx.x / kC;
  const int stride = LOOP ? (int)(gridDim.x / kC) : a.resident;   // distance to the job that follows on these SMs
  pdl_launch_dependents();
  pdl_wait();
  if (cluster_id >= a.lay.max_gather) return;                          // same decision in the whole cluster
  const uint4* job_list = reinterpret_cast<const uint4*>(a.ws + a.lay.gather);
  // the first job record is fetched together with the job count (the list has max_gather slots, so a record
  // read before the count is known is in bounds; the record at the mirrored position is the one that counts)
  const int n_jobs = min(a.ws[a.lay.header + H_NGATHER], a.lay.max_gather);
  int job_idx = n_jobs - 1 - cluster_id;
  if (job_idx < 0) return;

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  uint4* next_job = reinterpret_cast<uint4*>(smem + 32);                     // [2][4]
  float* part_all = reinterpret_cast<float*>(smem + 32 + 128);              // [2][kC][kR][rmax]
  float* mine = part_all + 2 * kC * kR * a.rmax;                             // [kR][rmax]
  float* v_sm = mine + kR * a.rmax;                                          // [kR][rmax]
  uint4* B_sm = reinterpret_cast<uint4*>(v_sm + kR * a.rmax);                // [rmax][per2max]
  const uint32_t bar = smem_u32(&bars[0]);        // completion of the B copies
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_init(smem_u32(&bars[1]), 1);             // arrival of the partial sums of all CTAs (even jobs of the loop)
    mbar_init(smem_u32(&bars[2]), 1);             // (odd jobs)
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  cluster_arrive();       // waited for right before the first remote store
  bool waited = false;

  int k = 0;              // jobs visited by this cluster
  int it_var = 0;         // jobs executed: parity of the partial-sum buffers and of the B barrier
  for (;; job_idx -= stride, ++k) {
    if (LOOP ? job_idx < 0 : k > 0) break;
    const int it = LOOP ? it_var : 0;
    GatherJob job;
    {
      uint4* dst = reinterpret_cast<uint4*>(&job);
      const uint4* jp = (LOOP && k > 0) ? next_job + (k & 1) * 4 : job_list + (size_t)job_idx * 4;
      dst[0] = jp[0]; dst[1] = jp[1]; dst[2] = jp[2]; dst[3] = jp[3];
    }
    const int next_idx = job_idx - stride;
    const bool has_next = stride > 0 && next_idx >= 0;
    // loop: the record of the following job is in flight while this job is reduced
    uint4 nrec = make_uint4(0, 0, 0, 0);
    if (LOOP && has_next && tid < 4) nrec = job_list[(size_t)next_idx * 4 + tid];

    int si = -1;
#pragma unroll
    for (int i = 0; i < kMaxSites; ++i)
      if (i < a.sites.n && a.sites.site[i].module == job.module) si = i;
    const int r = job.rank;
    const int n = min(job.count, kR);
    bool bad = r <= 0 || r > a.rmax || n <= 0 || !job.At || !job.B;
    int rows[kR];
#pragma unroll
    for (int t = 0; t < kR; ++t) {
      rows[t] = (t < n) ? job.rows[t] : -1;
      if (t < n && (rows[t] < 0 || rows[t] >= a.T)) bad = true;
    }
    if (si < 0 || bad) {
      // not a job of this launch's call sites, or a damaged record: every CTA of the cluster skips it alike
      if (si >= 0 && tid == 0 && crank == 0) atomicOr(a.err, ERR_BAD_ITEM);
      if (!LOOP) return;
      if (has_next && tid < 4) next_job[((k + 1) & 1) * 4 + tid] = nrec;
      __syncthreads();
      continue;
    }
    const ApplySite& site = a.sites.site[si];
    const int d1 = site.d1, d2 = site.d2;
    const int nv1 = d1 >> 3, nv2 = d2 >> 3;                 // 16-byte column groups per row
    const int per1 = (nv1 + kC - 1) / kC, per2 = (nv2 + kC - 1) / kC;
    const int lo1 = min((int)crank * per1, nv1), cnt1 = min(per1, nv1 - lo1);
    const int lo2 = min((int)crank * per2, nv2), cnt2 = min(per2, nv2 - lo2);
    const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(site.X);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(site.Y);
    const __nv_bfloat16* At = static_cast<const __nv_bfloat16*>(job.At);
    const char* Bslice = static_cast<const char*>(job.B) + (size_t)lo2 * 16;      // row j at + j * d2 * 2
    float* part = part_all + (size_t)(it & 1) * kC * kR * a.rmax;
    const uint32_t xbar = smem_u32(&bars[1 + (it & 1)]);
    const uint32_t xparity = (uint32_t)(it >> 1) & 1u, bparity = (uint32_t)it & 1u;

    // ---- everything the CTA will read is requested now: A^T and x into L2 (a cluster's first job; in the loop
    // the later ones were prefetched during the job before), B by bulk copies, y into registers ----
    {
      const size_t slice_bytes = (size_t)cnt1 * 16;
      const int n_lines = cnt1 > 0 ? (int)((slice_bytes + 127) / 128) + 1 : 0;
      if (k == 0) {
        prefetch_rows(reinterpret_cast<const char*>(At) + (size_t)lo1 * 16, (size_t)d1 * 2, r, slice_bytes, tid);
        if (!STAGE_B) prefetch_rows(Bslice, (size_t)d2 * 2, r, (size_t)cnt2 * 16, tid);
      }
      if (tid / kSegs < n) {            // kRowsPerPass >= kR: one group of kSegs threads per row of the job
        const int t = tid / kSegs;
        int row = rows[0];
#pragma unroll
        for (int q = 1; q < kR; ++q) row = (t == q) ? rows[q] : row;
        const char* p = reinterpret_cast<const char*>(X + (size_t)row * d1 + (size_t)lo1 * 8);
        for (int l = tid % kSegs; l < n_lines; l += kSegs) prefetch_l2(p + min((size_t)l * 128, slice_bytes - 16));
      }
    }
    if (tid == 0) mbar_expect_tx(xbar, (uint32_t)(kC * n * r) * 4u);
    if (STAGE_B) {
      if (warp == kThreads / 32 - 1) {
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)r * cnt2 * 16u);
        __syncwarp();
        if (cnt2 > 0) {
          for (int i = lane; i < r; i += 32)
            bulk_g2s(smem_u32(B_sm + (size_t)i * a.per2max), Bslice + (size_t)i * d2 * 2, cnt2 * 16, bar);
        }
      }
    }
    uint4 ypre[kYIter];
#pragma unroll
    for (int q4 = 0; q4 < kYIter; ++q4) {
      const int idx = tid + q4 * kThreads;
      ypre[q4] = make_uint4(0, 0, 0, 0);
      if (idx < n * cnt2) {
        const int t = idx / cnt2, g = idx % cnt2;
        int row = rows[0];
#pragma unroll
        for (int q = 1; q < kR; ++q) row = (t == q) ? rows[q] : row;
        ypre[q4] = *reinterpret_cast<const uint4*>(Y + (size_t)row * d2 + (size_t)(lo2 + g) * 8);
      }
    }

    // ---- shrink: partial v over this CTA's d1 slice, A^T straight from global memory -------------------
    const int seg = tid % kSegs;
    for (int j0 = 0; j0 < r; j0 += kRowsPerPass) {
      const int j = j0 + tid / kSegs;
      float acc[kR];
#pragma unroll
      for (int t = 0; t < kR; ++t) acc[t] = 0.f;
      if (j < r) {
        const __nv_bfloat16* arow = At + (size_t)j * d1 + (size_t)lo1 * 8;
        for (int v0 = seg; v0 < cnt1; v0 += kSegs * kUnroll) {
          uint4 aq[kUnroll];
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kSegs;
            aq[u] = (v < cnt1) ? ldg_stream(arow + (size_t)v * 8) : make_uint4(0, 0, 0, 0);
          }
#pragma unroll
          for (int t = 0; t < kR; ++t) {
            if (t < n) {
              const __nv_bfloat16* xrow = X + (size_t)rows[t] * d1 + (size_t)lo1 * 8;
              uint4 xq[kUnroll];
#pragma unroll
              for (int u = 0; u < kUnroll; ++u) {
                const int v = v0 + u * kSegs;
                xq[u] = (v < cnt1) ? *reinterpret_cast<const uint4*>(xrow + (size_t)v * 8) : make_uint4(0, 0, 0, 0);
              }
#pragma unroll
              for (int u = 0; u < kUnroll; ++u) {
                float av[8], xv[8];
                unpack8(aq[u], av);
                unpack8(xq[u], xv);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[t] = fmaf(xv[i], av[i], acc[t]);
              }
            }
          }
        }
      }
#pragma unroll
      for (int t = 0; t < kR; ++t) {
#pragma unroll
        for (int o = kSegs / 2; o > 0; o >>= 1) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], o);
      }
      if (seg == 0 && j < r) {
#pragma unroll
        for (int t = 0; t < kR; ++t) mine[t * a.rmax + j] = acc[t];
      }
    }
    if (LOOP && has_next && tid < 4) next_job[((k + 1) & 1) * 4 + tid] = nrec;
    __syncthreads();
    // The job that will run on these SMs next: its A^T and B slices are prefetched into L2 while this CTA waits
    // for the partial sums, so that its loads find L2 warm and HBM stays busy between two jobs.
    uint4 nj0 = make_uint4(0, 0, 0, 0), nj1 = nj0;
    if (has_next) {
      const uint4* np = LOOP ? next_job + ((k + 1) & 1) * 4 : job_list + (size_t)next_idx * 4;
      nj0 = np[0];
      nj1 = np[1];
    }
    if (!waited) {
      cluster_wait();       // every CTA of the cluster has started and initialised its barriers
      waited = true;
    }
    // hand this CTA's partial sums to every CTA of the cluster (slot `crank` of their `part`), one store per thread;
    // each store is counted on the receiver's barrier
    for (int idx = tid; idx < n * r * kC; idx += kThreads) {
      const int peer = idx % kC, e = idx / kC, t = e / r, j = e % r;
      st_async_f32(smem_u32(part + ((size_t)crank * kR + t) * a.rmax + j), xbar, (uint32_t)peer, mine[t * a.rmax + j]);
    }
    if (has_next) {
      const char* nAt = reinterpret_cast<const char*>(((uint64_t)nj0.y << 32) | nj0.x);
      const char* nB = reinterpret_cast<const char*>(((uint64_t)nj0.w << 32) | nj0.z);
      const int nr = (int)nj1.x, nmod = (int)nj1.z;
      int nsi = -1;
#pragma unroll
      for (int i = 0; i < kMaxSites; ++i)
        if (i < a.sites.n && a.sites.site[i].module == nmod) nsi = i;
      if (nsi >= 0 && nAt && nB && nr > 0 && nr <= a.rmax) {
        const int nd1 = a.sites.site[nsi].d1, nd2 = a.sites.site[nsi].d2;
        const int p1 = ((nd1 >> 3) + kC - 1) / kC, p2 = ((nd2 >> 3) + kC - 1) / kC;
        const int l1 = min((int)crank * p1, nd1 >> 3), c1 = min(p1, (nd1 >> 3) - l1);
        const int l2 = min((int)crank * p2, nd2 >> 3), c2 = min(p2, (nd2 >> 3) - l2);
        prefetch_rows(nAt + (size_t)l1 * 16, (size_t)nd1 * 2, nr, (size_t)c1 * 16, tid);
        prefetch_rows(nB + (size_t)l2 * 16, (size_t)nd2 * 2, nr, (size_t)c2 * 16, tid);
      }
    }
    // all kC x n x r partial sums have landed here; the peers wait for theirs likewise, so nobody is written after it left
    if (!mbar_wait(xbar, xparity)) {
      // A peer's partial sums never came.  This CTA's shared memory is still the target of the stores that are
      // missing, and of its own bulk copies: it stays for a second, equally bounded, wait on both before it leaves,
      // so that whatever is merely late has landed; a peer that is gone for good has raised the flag itself.
      if (tid == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
      mbar_wait(xbar, xparity);
      if (STAGE_B) mbar_wait(bar, bparity);
      return;
    }

    for (int idx = tid; idx < n * r; idx += kThreads) {
      const int t = idx / r, j = idx % r;
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < kC; ++c) sum += part[((size_t)c * kR + t) * a.rmax + j];
      v_sm[t * a.rmax + j] = sum * job.scale * job.gate[t];
    }
    __syncthreads();

    // ---- expand: this CTA's d2 slice ------------------------------------------------------------
    if (STAGE_B && !mbar_wait(bar, bparity)) {
      if (tid == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
      mbar_wait(bar, bparity);    // a second, equally bounded, chance for copies still in flight before leaving
      return;
    }
#pragma unroll
    for (int q4 = 0; q4 < kYIter; ++q4) {
      const int idx = tid + q4 * kThreads;
      if (idx < n * cnt2) {
        const int t = idx / cnt2, g = idx % cnt2;
        float out[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = 0.f;
        if (STAGE_B) {
          for (int j = 0; j < r; ++j) {
            float bv[8];
            unpack8(B_sm[(size_t)j * a.per2max + g], bv);
            const float vj = v_sm[t * a.rmax + j];
#pragma unroll
            for (int i = 0; i < 8; ++i) out[i] = fmaf(vj, bv[i], out[i]);
          }
        } else {
          // rank rows in batches of eight: independent loads (L2 hits) first, then the multiply-adds in rank order
          for (int j0 = 0; j0 < r; j0 += 8) {
            uint4 bq[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
              bq[u] = ldg_stream(Bslice + (size_t)min(j0 + u, r - 1) * d2 * 2 + (size_t)g * 16);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              if (j0 + u < r) {
                float bv[8];
                unpack8(bq[u], bv);
                const float vj = v_sm[t * a.rmax + j0 + u];
#pragma unroll
                for (int i = 0; i < 8; ++i) out[i] = fmaf(vj, bv[i], out[i]);
              }
            }
          }
        }
        float yv[8];
        unpack8(ypre[q4], yv);
#pragma unroll
        for (int i = 0; i < 8; ++i) yv[i] += out[i];
        int row = rows[0];
#pragma unroll
        for (int q = 1; q < kR; ++q) row = (t == q) ? rows[q] : row;
        *reinterpret_cast<uint4*>(Y + (size_t)row * d2 + (size_t)(lo2 + g) * 8) = pack8(yv);
      }
    }
    if (!LOOP) break;
    __syncthreads();        // B staging, mine and v are reused by the next job
    ++it_var;
  }
}

}  // namespace

milora_status launch_apply_decode_bf16(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                       cudaStream_t s) {
  (void)layer;
  if (ctx->desc.dtype != MILORA_BF16) return MILORA_E_SHAPE;
  DecodeArgs a;
  a.err = ctx->d_err;
  a.sites = sites;
  a.ws = g->ws_dev;
  a.lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  a.T = g->T;
  a.rmax = (ctx->desc.max_rank + 3) & ~3;
  int per2 = 0;
  for (int i = 0; i < sites.n; ++i) {
    const ApplySite& st = sites.site[i];
    if ((reinterpret_cast<uintptr_t>(st.X) & 15) || (reinterpret_cast<uintptr_t>(st.Y) & 15)) return MILORA_E_SHAPE;
    per2 = std::max(per2, (st.d2 / 8 + kC - 1) / kC);
  }
  if (kR * per2 > kYIter * kThreads) return MILORA_E_SHAPE;
  a.per2max = per2;
  const size_t smem_base = 32 + 128 + (size_t)(2 * kC + 2) * kR * a.rmax * sizeof(float);
  size_t smem = smem_base + (size_t)a.rmax * per2 * 16;
  // staging B pays only while four CTAs still fit on an SM (four is what the register budget allows)
  const bool stage_b = (smem + 1024) * 4 <= 227 * 1024;
  if (!stage_b) smem = smem_base;
  if (smem > 200 * 1024) return MILORA_E_SHAPE;
  void (*one_shot)(DecodeArgs) = stage_b ? decode_bf16_kernel<true, false> : decode_bf16_kernel<false, false>;
  void (*looped)(DecodeArgs) = stage_b ? decode_bf16_kernel<true, true> : decode_bf16_kernel<false, true>;
  int per_sm = 0;
  MILORA_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, one_shot, kThreads, smem));
  const int resident = std::max(1, ctx->sm_count * per_sm / kC);
  a.resident = resident;
  // One cluster per slot of the job list while the list is short; a list much longer than the GPU's capacity
  // (a mixed batch: slots are reserved for every row, most rows are prompt rows) is walked by resident clusters.
  // (Up to a few slots per resident cluster the one-shot kernel is the faster one: the hardware places its clusters
  // as SMs free up, which balances jobs of unequal size better than the loop's fixed stride.)
  const bool loop = a.lay.max_gather > 8 * resident;
  auto kernel = loop ? looped : one_shot;
  if (smem > 48 * 1024) {
    MILORA_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  }
  size_t grid = (size_t)(loop ? resident : a.lay.max_gather) * kC;
  if (grid > 0x7fffffffull) return MILORA_E_CAPACITY;
  MILORA_CUDA(ctx, launch_pdl(kernel, dim3((unsigned)grid), dim3(kThreads), smem, s, a));
  return MILORA_OK;
}

}  // namespace milora
