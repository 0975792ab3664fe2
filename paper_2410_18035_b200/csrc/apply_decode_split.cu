// Decode path of Eq. 1 for bf16 on sm_100a as two streaming kernels:
//   shrink:  v[job][t][j] = s * gate_t * sum_c x[row_t][c] * A^T[j][c]      (reads A^T once)
//   expand:  y[row_t][c] += sum_j v[job][t][j] * B[j][c]                      (reads B once, y once, writes y once)
// for the gathered rows of the decode work list (at most kGatherRows rows per job, all sharing one adapter).
//
// The cluster kernel of apply_decode_sm100.cu keeps one job inside one cluster, so a CTA runs a chain of
// dependent phases (its A^T slice, the exchange of partial sums, its B slice) and, once a step has more jobs
// than the GPU holds clusters, each generation of CTAs pays that chain again.  Here each kernel is a plain
// stream over small, equally sized units:
//   * a shrink unit is 16 rank rows x 1024 columns of A^T (32 KB); the partial products of the column chunks of
//     one job meet in the expand kernel, which adds them in chunk order;
//   * an expand unit is a 1024-column slice of B over all rank rows (32 KB at rank 16);
//   * both kernels are persistent (as many CTAs as the GPU holds) and take units from a counter, so unequal
//     units balance; the unit list runs from the heaviest modules (the list is ordered by module, and gate, up,
//     down come last) to the lightest;
//   * both contractions run as mma.sync m16n8k16 tiles fed from registers.  The path is bound by the adapter
//     stream, not by arithmetic: the point of the tensor cores here is the instruction count.  With scalar
//     multiply-adds a thread spends ~30 instructions (bf16 unpacking, one FMA per element and row) on every 16
//     bytes it loads, which the SMs cannot issue at HBM speed; an MMA consumes the packed bf16 words as loaded;
//   * the expand kernel is launched as a programmatic dependent of the shrink kernel: its CTAs start while the
//     shrink kernel drains, find their first unit and ask for its slice of B before they wait for v.
// v lives in a scratch buffer of the context.  Deterministic: fixed summation order in both kernels, the
// counters only decide which CTA computes a unit.
#include "milora_internal.h"

namespace milora {
namespace {

constexpr int kR = kGatherRows;
constexpr int kSThreads = 128;
constexpr int kSWarps = kSThreads / 32;
constexpr int kSRows = 16;         // rank rows per shrink unit: the M of one mma.sync tile
constexpr int kSCols = 1024;       // columns of A^T per shrink unit
constexpr int kSGroups = kSCols / 32 / kSWarps;   // 32-column groups a warp owns in a unit
constexpr int kSBatch = 4;         // groups whose loads a warp issues before it consumes them
constexpr int kEThreads = 128;
constexpr int kECols = 1024;       // columns of B per expand unit: four warps, four 64-column spans each
                                   // (512-column units: 52.1 us per layer on the 13B chain against 48.7)
constexpr int kMaxRankSplit = 256;

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 q;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
               : "l"(p));
  return q;
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ uint4 pack8(const float (&v)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

struct SplitArgs {
  int32_t* err;
  ApplySites sites;
  const int32_t* ws;
  milora_group_layout_t lay;
  int T;
  int rmax;                // floats per row of v
  int kcmax;               // column chunks of the widest d1 among the call sites
  float* v;                // [max_gather][kcmax][kR][rmax]: partial x . A^T per column chunk, scaled
  unsigned int* counters;  // [0] units handed out by the shrink kernel beyond the first per CTA, [1] by the expand kernel
};

// Rank rows of A^T per shrink unit.
__host__ __device__ inline int shrink_chunks(int d1) { return (d1 + kSCols - 1) / kSCols; }
__host__ __device__ inline int shrink_units(int d1, int rmax) { return ((rmax + kSRows - 1) / kSRows) * shrink_chunks(d1); }

// Units of the launch: module m owns units [base[m], base[m+1]); its jobs are first[m] + i, each cut into upj[m] units.
struct UnitMap {
  int base[MILORA_NMOD + 1];
  int first[MILORA_NMOD];
  int upj[MILORA_NMOD];
  int site[MILORA_NMOD];
};

template <bool EXPAND>
__device__ __forceinline__ void build_map(const SplitArgs& a, UnitMap* m, int tid) {
  if (tid == 0) {
    int off[MILORA_NMOD + 1];
#pragma unroll
    for (int i = 0; i <= MILORA_NMOD; ++i) off[i] = a.ws[a.lay.mod_gather_offset + i];
    const int n_jobs = max(0, min(a.ws[a.lay.header + H_NGATHER], a.lay.max_gather));
    int base = 0;
#pragma unroll
    for (int mod = 0; mod < MILORA_NMOD; ++mod) {
      const int lo = max(0, min(off[mod], n_jobs)), hi = max(lo, min(off[mod + 1], n_jobs));
      int si = -1;
      for (int i = 0; i < a.sites.n; ++i)
        if (a.sites.site[i].module == mod) si = i;
      int upj = 0;
      if (si >= 0) {
        if (EXPAND) {
          upj = (a.sites.site[si].d2 + kECols - 1) / kECols;
        } else {
          upj = shrink_units(a.sites.site[si].d1, a.rmax);
        }
      }
      m->first[mod] = lo;
      m->upj[mod] = upj;
      m->site[mod] = si;
      m->base[mod] = base;
      base += (hi - lo) * upj;
    }
    m->base[MILORA_NMOD] = base;
  }
  __syncthreads();
}

struct Unit {
  int job_idx, sub, site;
};
// Unit u counted from the end of the list (heaviest modules first).
__device__ __forceinline__ Unit find_unit(const UnitMap& m, int u) {
  const int ur = m.base[MILORA_NMOD] - 1 - u;
  int mod = 0;
#pragma unroll
  for (int i = 1; i < MILORA_NMOD; ++i)
    if (ur >= m.base[i]) mod = i;
  const int local = ur - m.base[mod], upj = m.upj[mod];
  Unit r;
  r.job_idx = m.first[mod] + local / upj;
  r.sub = local % upj;
  r.site = m.site[mod];
  return r;
}

__device__ __forceinline__ GatherJob load_job(const SplitArgs& a, int job_idx) {
  GatherJob job;
  const uint4* jp = reinterpret_cast<const uint4*>(a.ws + a.lay.gather) + (size_t)job_idx * 4;
  uint4* dst = reinterpret_cast<uint4*>(&job);
  dst[0] = jp[0]; dst[1] = jp[1]; dst[2] = jp[2]; dst[3] = jp[3];
  return job;
}
// The same test in both kernels, so that a damaged record is skipped by both.
__device__ __forceinline__ bool job_ok(const SplitArgs& a, const GatherJob& job, int site) {
  bool ok = site >= 0 && job.rank > 0 && job.rank <= a.rmax && job.count > 0 && job.At && job.B &&
            job.module == a.sites.site[site < 0 ? 0 : site].module;
#pragma unroll
  for (int t = 0; t < kR; ++t)
    if (t < job.count && (job.rows[t] < 0 || job.rows[t] >= a.T)) ok = false;
  return ok;
}

// L2 prefetch of `nrows` rows of `row_bytes` bytes, `pitch` bytes apart, spread over `nthreads` threads.
__device__ __forceinline__ void prefetch_rows(const char* base, size_t pitch, int nrows, int row_bytes, int tid, int nthreads) {
  if (row_bytes < 16 || nrows <= 0) return;
  const int lines = ((row_bytes + 127) >> 7) + 1;     // a row may start in the middle of a line
  for (int j = 0; j < nrows; ++j)
    for (int l = tid; l < lines; l += nthreads) prefetch_l2(base + (size_t)j * pitch + min(l * 128, row_bytes - 16));
}

// ---- shrink ---------------------------------------------------------------------------------------
// D (16 x 8, fp32) += A (16 x 16, bf16, row-major fragment) . B (16 x 8, bf16, column fragment)
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One unit: rank rows [j0, j0 + 16) of A^T against the job's rows of x over columns [kc * 1024, kc * 1024 + 1024).
// The contraction runs on the tensor cores only to save instructions (the kernel is bound by the A^T stream):
// M = rank rows, N = rows of x (up to 8, the job has at most 4), K = columns.  A thread (g = lane / 4, q = lane % 4)
// loads 16 bytes = 8 consecutive columns of rank rows g and g + 8 and of x row g, straight from global memory; the
// four 32-bit words of such a piece feed two MMAs as the k-pairs (2q, 2q+1) and (2q+8, 2q+9).  Which column
// stands behind which k is the same for both operands, and a sum does not care about the order of its terms.
__device__ __forceinline__ void shrink_unit(const SplitArgs& a, const GatherJob& job, int job_idx, const ApplySite& site,
                                            int sub, float (*red)[kSRows * 8], int tid) {
  const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, q = lane & 3;
  const int nv1 = site.d1 >> 3, r = job.rank, n = min(job.count, kR);
  const int chunks = shrink_chunks(site.d1);
  const int mb = sub / chunks, kc = sub % chunks, j0 = mb * kSRows;
  if (j0 >= r) return;
  // rank rows past the rank repeat the last one; their sums are dropped at the end
  const uint4* A0 = static_cast<const uint4*>(job.At) + (size_t)min(j0 + g, r - 1) * nv1;
  const uint4* A1 = static_cast<const uint4*>(job.At) + (size_t)min(j0 + g + 8, r - 1) * nv1;
  int xr = job.rows[0];
#pragma unroll
  for (int t = 1; t < kR; ++t) xr = (g == t) ? job.rows[t] : xr;
  const bool x_ok = g < n;
  const uint4* Xr = static_cast<const uint4*>(site.X) + (size_t)(x_ok ? xr : 0) * nv1;
  float c[4] = {0.f, 0.f, 0.f, 0.f};
  const int base = kc * (kSCols / 8) + warp * 4 + q;       // this thread's piece in the warp's first group
#pragma unroll
  for (int i0 = 0; i0 < kSGroups; i0 += kSBatch) {
    uint4 a0[kSBatch], a1[kSBatch], xq[kSBatch];
#pragma unroll
    for (int u = 0; u < kSBatch; ++u) {
      const int idx = base + (i0 + u) * (kSWarps * 4);
      const bool ok = idx < nv1;
      a0[u] = a1[u] = xq[u] = make_uint4(0, 0, 0, 0);
      if (ok) {
        a0[u] = ldg_stream(A0 + idx);
        a1[u] = ldg_stream(A1 + idx);
        if (x_ok) xq[u] = Xr[idx];
      }
    }
#pragma unroll
    for (int u = 0; u < kSBatch; ++u) {
      mma_16816(c, a0[u].x, a1[u].x, a0[u].y, a1[u].y, xq[u].x, xq[u].y);
      mma_16816(c, a0[u].z, a1[u].z, a0[u].w, a1[u].w, xq[u].z, xq[u].w);
    }
  }
  // accumulator fragment: c0, c1 = (rank row g, x rows 2q, 2q+1); c2, c3 = (rank row g + 8, same x rows)
  red[warp][g * 8 + 2 * q] = c[0];
  red[warp][g * 8 + 2 * q + 1] = c[1];
  red[warp][(g + 8) * 8 + 2 * q] = c[2];
  red[warp][(g + 8) * 8 + 2 * q + 1] = c[3];
  __syncthreads();
  {
    const int m = tid >> 3, t = tid & 7;       // kSThreads == kSRows * 8
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kSWarps; ++w) s += red[w][tid];
    float gt = job.gate[0];
#pragma unroll
    for (int i = 1; i < kR; ++i) gt = (t == i) ? job.gate[i] : gt;
    if (t < n && j0 + m < r)
      a.v[(((size_t)job_idx * a.kcmax + kc) * kR + t) * a.rmax + j0 + m] = s * job.scale * gt;
  }
  __syncthreads();
}

static_assert(kSThreads == kSRows * 8, "one thread per element of the 16 x 8 tile in the final sum");

__global__ void __launch_bounds__(kSThreads, 6) decode_shrink_kernel(SplitArgs a) {
  __shared__ UnitMap map;
  __shared__ float red[kSWarps][kSRows * 8];
  __shared__ int s_next[2];
  const int tid = threadIdx.x;
  // Nothing of the work list may be read before the kernels in front have completed.  The dependents are
  // released only after that wait: whatever runs of the expand kernel therefore runs after everything that
  // precedes this kernel on the stream, and may read the work list, B and y before its own wait.
  pdl_wait();
  if (blockIdx.x == 0 && tid == 0) a.counters[1] = 0;    // the expand kernel reads it after its wait
  pdl_launch_dependents();
  build_map<false>(a, &map, tid);
  const int total = map.base[MILORA_NMOD];
  // the first unit is the CTA's own index, the later ones come from the counter, fetched one unit ahead
  int u = blockIdx.x;
  for (int k = 0; u < total; ++k) {
    if (tid == 0) s_next[k & 1] = (int)gridDim.x + (int)atomicAdd(&a.counters[0], 1u);
    const Unit un = find_unit(map, u);
    const GatherJob job = load_job(a, un.job_idx);
    if (job_ok(a, job, un.site)) {
      shrink_unit(a, job, un.job_idx, a.sites.site[un.site], un.sub, red, tid);
    } else if (un.sub == 0 && tid == 0) {
      atomicOr(a.err, ERR_BAD_ITEM);
    }
    __syncthreads();
    u = s_next[k & 1];
  }
}

// ---- expand ---------------------------------------------------------------------------------------
// Tensor-core form of y[t][c] += sum_j v[t][j] B[j][c], again to save instructions: M = rows of the job (up to 4
// of the tile's 16), K = rank rows, N = columns.  The column fragment of the second operand wants the pair
// (B[j][c], B[j+1][c]) in one register while memory holds B row by row, so a thread loads 16 bytes = 8 columns of
// rank rows 2q, 2q+1, 2q+8, 2q+9 and interleaves them with byte permutes: eight MMAs then cover a 64-column span,
// the n-th column of MMA i being column 8n + i of the span.  With that numbering the accumulators of thread
// (g, q) are 16 consecutive columns of row g of y.  v enters as bf16 twice, as its rounded value and as the
// rounding remainder, which keeps the fp32 value of v to 2^-17.
constexpr int kESpan = 64;                                   // columns per group of eight MMAs
constexpr int kESpans = kECols / kESpan / (kEThreads / 32);          // spans a warp owns in a unit

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Four rank rows of one 16-row block for this thread's 8 columns.
struct BPiece {
  uint4 r0, r1, r8, r9;
};
__device__ __forceinline__ BPiece load_piece(const char* bcol, int kb, int q, int r, size_t pitch) {
  BPiece p;
  const int j = kb * 16 + 2 * q;
  p.r0 = ldg_stream(bcol + (size_t)min(j, r - 1) * pitch);
  p.r1 = ldg_stream(bcol + (size_t)min(j + 1, r - 1) * pitch);
  p.r8 = ldg_stream(bcol + (size_t)min(j + 8, r - 1) * pitch);
  p.r9 = ldg_stream(bcol + (size_t)min(j + 9, r - 1) * pitch);
  return p;
}
__device__ __forceinline__ void mma_piece(float (&acc)[8][4], const BPiece& p, const uint4 va) {
  const uint32_t w0[4] = {p.r0.x, p.r0.y, p.r0.z, p.r0.w}, w1[4] = {p.r1.x, p.r1.y, p.r1.z, p.r1.w};
  const uint32_t w8[4] = {p.r8.x, p.r8.y, p.r8.z, p.r8.w}, w9[4] = {p.r9.x, p.r9.y, p.r9.z, p.r9.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // columns 2i (low halves) and 2i + 1 (high halves) of the thread's eight
    const uint32_t b0e = __byte_perm(w0[i], w1[i], 0x5410), b1e = __byte_perm(w8[i], w9[i], 0x5410);
    const uint32_t b0o = __byte_perm(w0[i], w1[i], 0x7632), b1o = __byte_perm(w8[i], w9[i], 0x7632);
    mma_16816(acc[2 * i], va.x, 0u, va.y, 0u, b0e, b1e);
    mma_16816(acc[2 * i], va.z, 0u, va.w, 0u, b0e, b1e);
    mma_16816(acc[2 * i + 1], va.x, 0u, va.y, 0u, b0o, b1o);
    mma_16816(acc[2 * i + 1], va.z, 0u, va.w, 0u, b0o, b1o);
  }
}

// One unit: columns [sub * 1024, sub * 1024 + 1024) of B (all rank rows) into the job's rows of y.
// va_sm: the first operand's fragments, [rank block][lane] = {hi(k 2q,2q+1), hi(k 2q+8,2q+9), lo(..), lo(..)}.
__device__ __forceinline__ void expand_unit(const SplitArgs& a, const GatherJob& job, int job_idx, const ApplySite& site,
                                            int sub, float (*vs)[kMaxRankSplit], uint4 (*va_sm)[32], int tid) {
  const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, q = lane & 3;
  const int d2 = site.d2, nv2 = d2 >> 3, r = job.rank, n = min(job.count, kR);
  const int kblocks = (r + 15) >> 4;
  const size_t pitch = (size_t)d2 * 2;
  int yr = job.rows[0];
#pragma unroll
  for (int t = 1; t < kR; ++t) yr = (g == t) ? job.rows[t] : yr;
  const bool y_row_ok = g < n;
  uint4* Yrow = static_cast<uint4*>(site.Y) + (size_t)(y_row_ok ? yr : 0) * nv2;
  // The warp's spans and their rank blocks form one sequence of steps; the piece of step s + 1 is loaded before the
  // MMAs of step s, across span boundaries too, and the y pieces of the next span at the start of the current one,
  // so that the warp always has loads in flight.  The first piece and the first span's y go out before v is put
  // together, so that their latency and that of the chunk sums overlap.
  const int col8_0 = (sub * kECols + warp * kESpans * kESpan) >> 3;     // first span's start, in 8-column pieces
  const int nspans = max(0, min(kESpans, (nv2 - col8_0 + 7) >> 3));              // spans that start inside the matrix
  // this thread loads pieces col8 + g of a span and owns the results of its pieces col8 + 2q, col8 + 2q + 1
  auto piece_of = [&](int sp, int kb) {
    return load_piece(static_cast<const char*>(job.B) + (size_t)min(col8_0 + sp * 8 + g, nv2 - 1) * 16, kb, q, r, pitch);
  };
  auto y_of = [&](int sp, int which) {
    const int c = col8_0 + sp * 8 + 2 * q + which;
    return (y_row_ok && sp < nspans && c < nv2) ? Yrow[c] : make_uint4(0, 0, 0, 0);
  };
  BPiece cur;
  cur.r0 = cur.r1 = cur.r8 = cur.r9 = make_uint4(0, 0, 0, 0);
  if (nspans > 0) cur = piece_of(0, 0);
  uint4 y0 = y_of(0, 0), y1 = y_of(0, 1);
  // v = sum of the shrink kernel's partial products over the column chunks of d1, in chunk order
  {
    const int chunks = shrink_chunks(site.d1);
    for (int idx = tid; idx < n * r; idx += kEThreads) {
      const int t = idx / r, j = idx % r;
      // the loads of sixteen chunks go out together; the additions keep the chunk order
      const float* vp = a.v + (((size_t)job_idx * a.kcmax) * kR + t) * a.rmax + j;
      const size_t cstride = (size_t)kR * a.rmax;
      float sum = 0.f;
      for (int c0 = 0; c0 < chunks; c0 += 16) {
        float part[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) part[i] = (c0 + i < chunks) ? vp[(size_t)(c0 + i) * cstride] : 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += part[i];
      }
      vs[t][j] = sum;
    }
  }
  __syncthreads();
  for (int idx = tid; idx < kblocks * 32; idx += kEThreads) {
    const int kb = idx >> 5, l = idx & 31, gg = l >> 2, qq = l & 3;
    float v4[4] = {0.f, 0.f, 0.f, 0.f};
    if (gg < n) {
      const int j = kb * 16 + 2 * qq;
      if (j < r) v4[0] = vs[gg][j];
      if (j + 1 < r) v4[1] = vs[gg][j + 1];
      if (j + 8 < r) v4[2] = vs[gg][j + 8];
      if (j + 9 < r) v4[3] = vs[gg][j + 9];
    }
    uint4 f;
    f.x = pack_bf16(v4[0], v4[1]);
    f.y = pack_bf16(v4[2], v4[3]);
    f.z = pack_bf16(v4[0] - bf16_lo(f.x), v4[1] - bf16_hi(f.x));
    f.w = pack_bf16(v4[2] - bf16_lo(f.y), v4[3] - bf16_hi(f.y));
    va_sm[kb][l] = f;
  }
  __syncthreads();
  if (nspans > 0) {
#pragma unroll 1
    for (int sp = 0; sp < nspans; ++sp) {
      const int col8 = col8_0 + sp * 8;
      const uint4 yn0 = y_of(sp + 1, 0), yn1 = y_of(sp + 1, 1);
      float acc[8][4];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
#pragma unroll 1
      for (int kb = 0; kb < kblocks; ++kb) {
        BPiece nxt = cur;
        if (kb + 1 < kblocks) nxt = piece_of(sp, kb + 1);
        else if (sp + 1 < nspans) nxt = piece_of(sp + 1, 0);
        mma_piece(acc, cur, va_sm[kb][lane]);
        cur = nxt;
      }
      // acc[i][0] is column 16q + i of the span, acc[i][1] column 16q + 8 + i, both of row g
      if (y_row_ok && col8 + 2 * q < nv2) {
        const uint32_t w[4] = {y0.x, y0.y, y0.z, y0.w};
        float o[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          o[2 * i] = bf16_lo(w[i]) + acc[2 * i][0];
          o[2 * i + 1] = bf16_hi(w[i]) + acc[2 * i + 1][0];
        }
        Yrow[col8 + 2 * q] = pack8(o);
      }
      if (y_row_ok && col8 + 2 * q + 1 < nv2) {
        const uint32_t w[4] = {y1.x, y1.y, y1.z, y1.w};
        float o[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          o[2 * i] = bf16_lo(w[i]) + acc[2 * i][1];
          o[2 * i + 1] = bf16_hi(w[i]) + acc[2 * i + 1][1];
        }
        Yrow[col8 + 2 * q + 1] = pack8(o);
      }
      y0 = yn0;
      y1 = yn1;
    }
  }
  __syncthreads();    // vs and va_sm are rewritten by the next unit
}

__global__ void __launch_bounds__(kEThreads, 4) decode_expand_kernel(SplitArgs a) {
  __shared__ UnitMap map;
  __shared__ float vs[kR][kMaxRankSplit];
  __shared__ uint4 va_sm[kMaxRankSplit / 16][32];
  __shared__ int s_next[2];
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  // The shrink kernel released this grid after its own wait, so the work list, the adapters and y are final
  // here; only v and the unit counter have to wait for the shrink kernel to complete.  Until then the CTA finds
  // its first unit and asks for that unit's slice of B.
  build_map<true>(a, &map, tid);
  const int total = map.base[MILORA_NMOD];
  int u = blockIdx.x;
  if (u < total) {
    const Unit un = find_unit(map, u);
    const GatherJob job = load_job(a, un.job_idx);
    if (job_ok(a, job, un.site)) {
      const ApplySite& st = a.sites.site[un.site];
      const int c0 = un.sub * kECols;
      prefetch_rows(static_cast<const char*>(job.B) + (size_t)c0 * 2, (size_t)st.d2 * 2, job.rank,
                    min(kECols * 2, (st.d2 - c0) * 2), tid, kEThreads);
    }
  }
  pdl_wait();
  if (blockIdx.x == 0 && tid == 0) a.counters[0] = 0;    // the next shrink kernel starts from zero
  for (int k = 0; u < total; ++k) {
    if (tid == 0) s_next[k & 1] = (int)gridDim.x + (int)atomicAdd(&a.counters[1], 1u);
    const Unit un = find_unit(map, u);
    const GatherJob job = load_job(a, un.job_idx);
    if (job_ok(a, job, un.site)) expand_unit(a, job, un.job_idx, a.sites.site[un.site], un.sub, vs, va_sm, tid);
    __syncthreads();
    u = s_next[k & 1];
  }
}

}  // namespace

milora_status launch_apply_decode_split(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                        cudaStream_t s) {
  (void)layer;
  if (ctx->desc.dtype != MILORA_BF16) return MILORA_E_SHAPE;
  SplitArgs a;
  a.err = ctx->d_err;
  a.sites = sites;
  a.ws = g->ws_dev;
  a.lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  a.T = g->T;
  a.rmax = (ctx->desc.max_rank + 3) & ~3;
  if (a.rmax > kMaxRankSplit) return MILORA_E_SHAPE;
  int upj_s = 1, upj_e = 1, kcmax = 1;
  for (int i = 0; i < sites.n; ++i) {
    const ApplySite& st = sites.site[i];
    if ((reinterpret_cast<uintptr_t>(st.X) & 15) || (reinterpret_cast<uintptr_t>(st.Y) & 15)) return MILORA_E_SHAPE;
    if ((st.d1 & 7) || (st.d2 & 7)) return MILORA_E_SHAPE;
    upj_s = std::max(upj_s, shrink_units(st.d1, a.rmax));
    kcmax = std::max(kcmax, shrink_chunks(st.d1));
    upj_e = std::max(upj_e, (st.d2 + kECols - 1) / kECols);
  }
  if (a.lay.max_gather < 1) return MILORA_OK;
  // scratch: 64 floats of counters, then v
  a.kcmax = kcmax;
  const size_t need = 64 + (size_t)a.lay.max_gather * kcmax * kR * a.rmax;
  if (need * sizeof(float) > ((size_t)256 << 20)) return MILORA_E_SHAPE;
  if (need > ctx->dsplit_floats) {
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    if (ctx->d_dsplit) MILORA_CUDA(ctx, cudaFree(ctx->d_dsplit));
    ctx->d_dsplit = nullptr;
    ctx->dsplit_floats = 0;
    MILORA_CUDA(ctx, cudaMalloc(&ctx->d_dsplit, need * sizeof(float)));
    ctx->dsplit_floats = need;
    ctx->dsplit_dirty = true;
  }
  if (ctx->dsplit_dirty) {
    // both counters start from zero; afterwards each kernel leaves the other's counter at zero for the next call
    MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_dsplit, 0, 64 * sizeof(float), s));
  }
  a.counters = reinterpret_cast<unsigned int*>(ctx->d_dsplit);
  a.v = ctx->d_dsplit + 64;
  if (ctx->dsplit_occ_s == 0) {
    MILORA_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctx->dsplit_occ_s, decode_shrink_kernel, kSThreads, 0));
    MILORA_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ctx->dsplit_occ_e, decode_expand_kernel, kEThreads, 0));
    if (ctx->dsplit_occ_s < 1 || ctx->dsplit_occ_e < 1) return MILORA_E_CUDA;
  }
  const long long cap_s = (long long)ctx->sm_count * ctx->dsplit_occ_s, cap_e = (long long)ctx->sm_count * ctx->dsplit_occ_e;
  const long long grid_s = std::min(cap_s, (long long)a.lay.max_gather * upj_s);
  const long long grid_e = std::min(cap_e, (long long)a.lay.max_gather * upj_e);
  // if the second launch fails the counters are not back at zero: clear them on the next call
  ctx->dsplit_dirty = true;
  MILORA_CUDA(ctx, launch_pdl(decode_shrink_kernel, dim3((unsigned)grid_s), dim3(kSThreads), 0, s, a));
  MILORA_CUDA(ctx, launch_pdl(decode_expand_kernel, dim3((unsigned)grid_e), dim3(kEThreads), 0, s, a));
  ctx->dsplit_dirty = false;
  return MILORA_OK;
}

}  // namespace milora
