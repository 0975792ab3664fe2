// Decode path of Eq. 1 for bf16 on sm_100a as ONE persistent launch over any number of layers:
//   shrink:  v[job][t][j]  = s * gate_t * sum_c x[row_t][c] * A^T[j][c]
//   expand:  y[row_t][c]  += sum_j v[job][t][j] * B[j][c]
// for the gathered rows of the decode work lists (at most kGatherRows rows per job, all sharing one adapter;
// Section 3.3: the route is fixed per request, so the lists stay valid from step to step).
//
// Shape of the kernel
//   * One CTA per SM, kWarps independent worker warps per CTA.  A worker owns kBufs shared-memory buffers and runs
//     its own software pipeline: it asks for the next piece of adapter (a "stage": up to kStageBytes of the A or B
//     operand image, one contiguous cp.async.bulk, plus the job's rows of x or y, one bulk copy per row) while it
//     computes on the one that has arrived.  Workers never synchronise with each other inside the CTA.
//   * Work is cut into units: `unit_stages` consecutive stages of one job's shrink or expand.  Units are numbered
//     so that every shrink unit of a job precedes all of its expand units, and the expand units of layer l come
//     after the shrink units of layer l + 1.  The first units are assigned by worker index, later ones come from a
//     counter (fetched ahead), so unequal units balance.
//   * A shrink unit leaves its partial x . A^T in global scratch and counts itself on the job; the unit that
//     arrives last adds the partials in unit order (deterministic), applies scale and gate, and publishes v as
//     ready-made mma.sync fragments (bf16 value + bf16 remainder, i.e. v to 2^-17).  An expand unit waits
//     (bounded) for that flag.  Since units are handed out in order and a worker issues its units in order, the
//     unit with the smallest number that is not finished can always proceed: no deadlock while all CTAs are
//     resident (grid = number of SMs, one CTA per SM).
//   * Both contractions run on mma.sync m16n8k16 fed by ldmatrix from the operand images (the images are
//     8 x 16-byte core matrices, exactly what ldmatrix reads without bank conflicts).  The path is bound by the
//     adapter stream; the tensor cores are used for the instruction count.
//     shrink: M = rank rows, N = rows of x, K = columns of d1.
//     expand: M = columns of d2, N = (row t, value | remainder), K = rank rows; y is updated in shared memory and
//     written back with one bulk store per row.
//   * The job states and the unit counter clean themselves up (last expand unit of a job, last worker of the grid),
//     so a launch leaves the scratch ready for the next one.
#include <algorithm>
#include <cstring>

#include "milora_internal.h"
#include "sm100_ptx.cuh"

namespace milora {
namespace {

using namespace ptx;

constexpr int kR = kGatherRows;
constexpr int kWarps = 5;                        // worker warps per CTA
constexpr int kBufs = 2;                         // buffers (stages in flight) per worker
constexpr int kThreads = kWarps * 32;
constexpr int kStageBytes = 16384;               // adapter bytes per stage
constexpr int kRowBytesMax = kStageBytes / 16;   // a row of x / y per stage: cols * 2 bytes, cols <= kStageBytes / 32
constexpr int kRowPad = 16;                      // keeps the rows of one stage on different banks
constexpr int kBufBytes = kStageBytes + kR * (kRowBytesMax + kRowPad);
constexpr int kBufStride = (kBufBytes + 127) & ~127;
constexpr int kStaticRounds = 2;                 // units per worker assigned by index before the counter is used
constexpr int kUnitRing = 4;                     // unit records a worker keeps (issue runs ahead of compute)
constexpr int kMaxSeg = 2 * kMaxStreamLayers * MILORA_NMOD;
constexpr uint32_t kReady = 0x80000000u;
constexpr uint32_t kDepSpin = 1u << 22;          // polls of a job's ready flag before an expand unit gives up

struct StreamArgs {
  int32_t* err;
  const StreamLayer* layers;   // device array, or nullptr: `one` is the only layer
  StreamLayer one;
  int n_layers;
  int d1[MILORA_NMOD], d2[MILORA_NMOD];
  int rp;                      // rank pad of the context: fixes the columns per stage
  int cols;                    // columns of d1 / d2 per stage
  int unit_stages;             // stages per unit
  int kcmax;                   // most shrink units per job over the modules
  uint32_t* ctrl;              // [0] units handed out beyond the static rounds, [1] workers that have finished
  uint32_t* job_state;         // [jobs][2]: shrink units arrived | kReady, expand units done
  float* partial;              // [jobs][kcmax][kR][rp]
  uint2* vfrag;                // [jobs][rp / 16][32]
};

struct UnitRec {               // what a worker needs to know about a unit, in shared memory
  const char* img;             // operand image of the phase (A image for shrink, B image for expand)
  const char* rows_base;       // X or Y of the module
  int32_t rows[kR];
  float gate[kR];
  float scale;
  int32_t n, rp, rank;
  int32_t d, phase, module;
  int32_t stage0, n_stages;    // stage range of the job's phase covered by this unit
  int32_t job, sub, upj_s, upj_e;
  int32_t ok;
};

struct Smem {
  StreamLayer layers[kMaxStreamLayers];
  int32_t seg_base[kMaxSeg + 1];
  int32_t first[kMaxStreamLayers][MILORA_NMOD + 1];
  int32_t upj[2][MILORA_NMOD];
  UnitRec unit[kWarps][kUnitRing];
  float vsum[kWarps][kR][kImagePadMax];
  uint64_t full[kWarps][kBufs];
  int32_t buf_unit[kWarps][kBufs], buf_stage[kWarps][kBufs];
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts16(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Position p of the queue -> (layer of the launch, phase).  Order: S0, then S_l, E_{l-1} for l = 1..L-1, then E_{L-1}.
__device__ __forceinline__ void pos_to_layer(int p, int L, int* li, int* phase) {
  if (p == 0) { *li = 0; *phase = 0; }
  else if (p == 2 * L - 1) { *li = L - 1; *phase = 1; }
  else if (p & 1) { *li = (p + 1) >> 1; *phase = 0; }
  else { *li = (p >> 1) - 1; *phase = 1; }
}

// ---- unit look-up ------------------------------------------------------------------------------------
// Fills `r` for unit u (all lanes compute the same values; lanes 0..3 fetch the 64-byte job record).
__device__ __forceinline__ void decode_unit(const StreamArgs& a, const Smem& sm, int n_seg, int u, UnitRec* r, int lane) {
  // segment = (queue position, module): binary search over the prefix table
  int lo = 0, hi = n_seg;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (sm.seg_base[mid] <= u) lo = mid; else hi = mid;
  }
  const int p = lo / MILORA_NMOD, m = lo % MILORA_NMOD;
  int li, phase;
  pos_to_layer(p, a.n_layers, &li, &phase);
  const int local = u - sm.seg_base[lo];
  const int upj = sm.upj[phase][m];
  const int job_local = sm.first[li][m] + local / upj, sub = local % upj;
  const StreamLayer& L = sm.layers[li];
  // the job record: four 16-byte pieces, one per lane, then handed around the warp
  const uint4* jp = reinterpret_cast<const uint4*>(L.ws + L.off_gather) + (size_t)job_local * (kJobInts / 4);
  uint4 piece = make_uint4(0, 0, 0, 0);
  if (lane < 4) piece = jp[lane];
  GatherJob job;
  uint32_t* jw = reinterpret_cast<uint32_t*>(&job);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    jw[4 * i + 0] = __shfl_sync(0xffffffffu, piece.x, i);
    jw[4 * i + 1] = __shfl_sync(0xffffffffu, piece.y, i);
    jw[4 * i + 2] = __shfl_sync(0xffffffffu, piece.z, i);
    jw[4 * i + 3] = __shfl_sync(0xffffffffu, piece.w, i);
  }
  const int d1 = a.d1[m], d2 = a.d2[m];
  const int rpj = (job.rank + 15) & ~15;
  bool ok = job.rank > 0 && rpj <= a.rp && job.count > 0 && job.count <= kR && job.At != nullptr && job.module == m &&
            L.X[m] != nullptr && L.Y[m] != nullptr;
#pragma unroll
  for (int t = 0; t < kR; ++t)
    if (t < job.count && (job.rows[t] < 0 || job.rows[t] >= L.T)) ok = false;
  if (lane == 0) {
    const int d = phase ? d2 : d1;
    const int stages = (d + a.cols - 1) / a.cols;
    const AdapterLayout al = adapter_layout(d1, d2, ok ? job.rank : 1, 2);
    r->img = static_cast<const char*>(job.At) + (phase ? al.off_b_img : al.off_a_img);
    r->rows_base = static_cast<const char*>(phase ? L.Y[m] : L.X[m]);
#pragma unroll
    for (int t = 0; t < kR; ++t) { r->rows[t] = job.rows[t]; r->gate[t] = job.gate[t]; }
    r->scale = job.scale;
    r->n = job.count; r->rp = rpj; r->rank = job.rank;
    r->d = d; r->phase = phase; r->module = m;
    r->stage0 = sub * a.unit_stages;
    r->n_stages = min(a.unit_stages, stages - sub * a.unit_stages);
    r->job = L.job_base + job_local; r->sub = sub;
    r->upj_s = sm.upj[0][m]; r->upj_e = sm.upj[1][m];
    r->ok = ok ? 1 : 0;
  }
}

// ---- issue: the copies of one stage -------------------------------------------------------------------
// Lane 0 only.  buf: shared address of the buffer; bar: its mbarrier.
__device__ __forceinline__ void issue_stage(const StreamArgs& a, const UnitRec& r, int stage_in_unit, uint32_t buf, uint32_t bar,
                                            bool rows_too) {
  const int c0 = (r.stage0 + stage_in_unit) * a.cols;
  const int ncols = min(a.cols, r.d - c0);
  // both images are contiguous in column order: rp * 2 bytes per column
  const uint32_t bytes_img = (uint32_t)ncols * r.rp * 2;
  const uint32_t bytes_row = (uint32_t)ncols * 2;
  if (!rows_too) {
    mbar_expect_tx(bar, bytes_img + (uint32_t)r.n * bytes_row);
    bulk_g2s(buf, r.img + (size_t)c0 * r.rp * 2, bytes_img, bar);
  } else {
    const uint32_t rstride = (uint32_t)a.cols * 2 + kRowPad;
    for (int t = 0; t < r.n; ++t)
      bulk_g2s(buf + kStageBytes + t * rstride, r.rows_base + ((size_t)r.rows[t] * r.d + c0) * 2, bytes_row, bar);
  }
}

// ---- shrink: one stage into the unit's accumulators ---------------------------------------------------------
// acc[jb] is the 16 x 8 tile (rank rows jb*16.., rows of x) of this lane: c0, c1 = (rank row g, x rows 2q, 2q+1),
// c2, c3 = (rank row g + 8, same x rows).
__device__ __forceinline__ void shrink_stage(const StreamArgs& a, const UnitRec& r, int stage_in_unit, uint32_t buf,
                                             float (&acc)[kImagePadMax / 16][4], int lane) {
  const int g = lane >> 2, q = lane & 3, mi = lane >> 3;
  const int c0 = (r.stage0 + stage_in_unit) * a.cols;
  const int ncols = min(a.cols, r.d - c0);
  const int rp = r.rp, jblocks = rp >> 4;
  const uint32_t rstride = (uint32_t)a.cols * 2 + kRowPad;
  const bool x_ok = g < r.n;
  const uint32_t xrow = buf + kStageBytes + (x_ok ? g : 0) * rstride + 4 * q;
  // ldmatrix row address of this lane inside a 64-column chunk, for k step 0 and rank block 0
  const uint32_t lane_off = (uint32_t)(((mi >> 1) * (rp >> 3) + (mi & 1)) * 128 + (lane & 7) * 16);
  for (int kc = 0; kc < (ncols >> 6); ++kc) {
    const uint32_t chunk = buf + (uint32_t)kc * rp * 128 + lane_off;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      uint32_t b0 = 0, b1 = 0;
      if (x_ok) {
        b0 = lds32(xrow + (kc * 64 + s * 16) * 2);
        b1 = lds32(xrow + (kc * 64 + s * 16 + 8) * 2);
      }
#pragma unroll
      for (int jb = 0; jb < kImagePadMax / 16; ++jb) {
        if (jb < jblocks) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4(chunk + (uint32_t)((2 * s) * (rp >> 3) + 2 * jb) * 128, a0, a1, a2, a3);
          mma_16816(acc[jb], a0, a1, a2, a3, b0, b1);
        }
      }
    }
  }
}

// End of a shrink unit: partial products to scratch, count on the job; the last unit of the job adds them up in
// unit order and publishes v as the fragments of the expand MMAs.
__device__ __forceinline__ void shrink_finish(const StreamArgs& a, const UnitRec& r, float (&acc)[kImagePadMax / 16][4],
                                              float (*vsum)[kImagePadMax], int lane) {
  const int g = lane >> 2, q = lane & 3;
  const int rp = r.rp, jblocks = rp >> 4;
  float* part = a.partial + ((size_t)r.job * a.kcmax + r.sub) * kR * a.rp;
  if (q < 2) {
#pragma unroll
    for (int jb = 0; jb < kImagePadMax / 16; ++jb) {
      if (jb < jblocks) {
        const int j = jb * 16 + g;
        part[(2 * q) * a.rp + j] = acc[jb][0];
        part[(2 * q + 1) * a.rp + j] = acc[jb][1];
        part[(2 * q) * a.rp + j + 8] = acc[jb][2];
        part[(2 * q + 1) * a.rp + j + 8] = acc[jb][3];
      }
    }
  }
  __syncwarp();
  uint32_t* state = a.job_state + 2 * (size_t)r.job;
  uint32_t old = 0;
  if (lane == 0) {
    __threadfence();
    old = atomicAdd(state, 1u);
    __threadfence();
  }
  old = __shfl_sync(0xffffffffu, old, 0);
  if (old != (uint32_t)r.upj_s - 1) return;
  // this unit arrived last: every partial of the job is visible now
  const float* base = a.partial + (size_t)r.job * a.kcmax * kR * a.rp;
  const size_t ustride = (size_t)kR * a.rp;
  for (int idx = lane; idx < kR * rp; idx += 32) {
    const int t = idx / rp, j = idx % rp;
    const float* vp = base + t * a.rp + j;
    float sum = 0.f;
    for (int c0 = 0; c0 < r.upj_s; c0 += 8) {
      float p8[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) p8[i] = (c0 + i < r.upj_s) ? __ldcg(vp + (size_t)(c0 + i) * ustride) : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) sum += p8[i];
    }
    vsum[t][j] = (t < r.n) ? sum * r.scale * r.gate[t] : 0.f;
  }
  __syncwarp();
  // fragment of the second MMA operand (K = rank rows, N = 8): column n = g holds row t = g / 2 of v, its bf16
  // value for even g and the remainder after that rounding for odd g
  {
    const int t = g >> 1;
    const bool rem = g & 1;
    uint2* out = a.vfrag + (size_t)r.job * (a.rp >> 4) * 32;
    for (int ks = 0; ks < jblocks; ++ks) {
      float v4[4] = {vsum[t][ks * 16 + 2 * q], vsum[t][ks * 16 + 2 * q + 1], vsum[t][ks * 16 + 2 * q + 8],
                     vsum[t][ks * 16 + 2 * q + 9]};
      uint32_t w0 = pack_bf16(v4[0], v4[1]), w1 = pack_bf16(v4[2], v4[3]);
      if (rem) {
        const uint32_t h0 = w0, h1 = w1;
        w0 = pack_bf16(v4[0] - bf16_lo(h0), v4[1] - bf16_hi(h0));
        w1 = pack_bf16(v4[2] - bf16_lo(h1), v4[3] - bf16_hi(h1));
      }
      out[ks * 32 + lane] = make_uint2(w0, w1);
    }
  }
  __syncwarp();
  if (lane == 0) {
    __threadfence();
    st_release(state, kReady);
  }
}

// ---- expand: one stage, y updated in shared memory and stored back --------------------------------------------
__device__ __forceinline__ void expand_stage(const StreamArgs& a, const UnitRec& r, int stage_in_unit, uint32_t buf,
                                             const uint2 (&vb)[kImagePadMax / 16], int lane) {
  const int g = lane >> 2, q = lane & 3, mi = lane >> 3;
  const int c0 = (r.stage0 + stage_in_unit) * a.cols;
  const int ncols = min(a.cols, r.d - c0);
  const int rp = r.rp, ksteps = rp >> 4;
  const uint32_t rstride = (uint32_t)a.cols * 2 + kRowPad;
  const bool row_ok = q < r.n;
  const uint32_t yrow = buf + kStageBytes + (row_ok ? q : 0) * rstride + 2 * g;
  // ldmatrix row address inside a 128-column block for rank step 0, column step 0:
  // core matrix (n / 8, k / 8) at ((k / 8) * 16 + n / 8) * 128
  const uint32_t lane_off = (uint32_t)(((mi >> 1) * 16 + (mi & 1)) * 128 + (lane & 7) * 16);
  for (int nb = 0; nb < (ncols >> 7); ++nb) {
    const uint32_t blk = buf + (uint32_t)nb * rp * 256 + lane_off;
#pragma unroll
    for (int ns = 0; ns < 8; ++ns) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < kImagePadMax / 16; ++ks) {
        if (ks < ksteps) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4(blk + (uint32_t)((2 * ks) * 16 + 2 * ns) * 128, a0, a1, a2, a3);
          mma_16816(c, a0, a1, a2, a3, vb[ks].x, vb[ks].y);
        }
      }
      // c0 + c1: column g of the step, row t = q (value part + remainder part); c2 + c3: column g + 8
      if (row_ok) {
        const uint32_t p = yrow + (nb * 128 + ns * 16) * 2;
        const float y0 = __uint_as_float(lds16(p) << 16) + (c[0] + c[1]);
        const float y1 = __uint_as_float(lds16(p + 16) << 16) + (c[2] + c[3]);
        sts16(p, __bfloat16_as_ushort(__float2bfloat16_rn(y0)));
        sts16(p + 16, __bfloat16_as_ushort(__float2bfloat16_rn(y1)));
      }
    }
  }
  fence_proxy_async_smem();
  __syncwarp();
  if (lane == 0) {
    for (int t = 0; t < r.n; ++t)
      bulk_s2g(const_cast<char*>(r.rows_base) + ((size_t)r.rows[t] * r.d + c0) * 2, buf + kStageBytes + t * rstride,
               (uint32_t)ncols * 2);
    bulk_commit_group();
  }
}

// ---- the kernel --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1) decode_stream_kernel(StreamArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw + (size_t)kWarps * kBufs * kBufStride);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = a.n_layers;
  const int n_seg = 2 * L * MILORA_NMOD;
  if (tid == 0) {
    for (int w = 0; w < kWarps; ++w)
      for (int b = 0; b < kBufs; ++b) mbar_init(smem_u32(&sm.full[w][b]), 1);
    fence_barrier_init();
  }
  pdl_launch_dependents();
  pdl_wait();

  // ---- layer records and the unit table (every CTA builds the same one) ----
  {
    const uint4* src = reinterpret_cast<const uint4*>(a.layers ? a.layers : &a.one);
    uint4* dst = reinterpret_cast<uint4*>(sm.layers);
    if (a.layers) {
      for (int i = tid; i < L * (int)(sizeof(StreamLayer) / 16); i += kThreads) dst[i] = src[i];
    } else if (tid == 0) {
      sm.layers[0] = a.one;
    }
    if (tid < MILORA_NMOD) {
      const int ss = (a.d1[tid] + a.cols - 1) / a.cols, se = (a.d2[tid] + a.cols - 1) / a.cols;
      sm.upj[0][tid] = (ss + a.unit_stages - 1) / a.unit_stages;
      sm.upj[1][tid] = (se + a.unit_stages - 1) / a.unit_stages;
    }
  }
  __syncthreads();
  for (int i = tid; i < L * (MILORA_NMOD + 1); i += kThreads) {
    const int li = i / (MILORA_NMOD + 1), m = i % (MILORA_NMOD + 1);
    const StreamLayer& Ly = sm.layers[li];
    const int n_jobs = max(0, min(Ly.ws[Ly.off_header + H_NGATHER], Ly.max_gather));
    sm.first[li][m] = max(0, min(Ly.ws[Ly.off_mod_gather + m], n_jobs));
  }
  __syncthreads();
  for (int i = tid; i < n_seg; i += kThreads) {
    const int p = i / MILORA_NMOD, m = i % MILORA_NMOD;
    int li, phase;
    pos_to_layer(p, L, &li, &phase);
    const StreamLayer& Ly = sm.layers[li];
    int cnt = max(0, sm.first[li][m + 1] - sm.first[li][m]) * sm.upj[phase][m];
    if (Ly.X[m] == nullptr || Ly.Y[m] == nullptr) cnt = 0;
    sm.seg_base[i + 1] = cnt;       // counts first, prefix sums below
  }
  __syncthreads();
  if (warp == 0) {
    // inclusive scan of seg_base[1..n_seg] by one warp, 32 entries per pass
    int carry = 0;
    for (int b = 0; b < n_seg; b += 32) {
      const int i = b + lane;
      int v = (i < n_seg) ? sm.seg_base[i + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
      }
      if (i < n_seg) sm.seg_base[i + 1] = carry + v;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
    if (lane == 0) sm.seg_base[0] = 0;
  }
  __syncthreads();
  const int total = sm.seg_base[n_seg];

  // ---- worker ----
  const int n_workers = (int)gridDim.x * kWarps;
  const int wid = warp * (int)gridDim.x + (int)blockIdx.x;     // neighbouring units go to different SMs
  const uint32_t buf0 = smem_u32(smem_raw) + (uint32_t)(warp * kBufs) * kBufStride;
  UnitRec* ring = sm.unit[warp];
  int n_fetched = 0;              // units this worker has taken so far
  int n_kept = 0;                 // ... of which were valid (they take turns in the ring of unit records)
  int n_issued = 0, n_done = 0;   // stages issued / consumed (buffer = count % kBufs, parity = (count / kBufs) & 1)
  int iu = -1, is = 0;            // ring index and next stage of the unit being issued (-1: none)
  bool dry = false, failed = false;
  uint32_t next_dyn = 0;          // counter value fetched ahead
  bool have_dyn = false;
  float acc[kImagePadMax / 16][4];
  uint2 vb[kImagePadMax / 16];
  int cu_loaded = -1;             // ring index of the unit whose fragments are in vb

  auto take_unit = [&]() {
    // next unit of this worker into the ring; sets iu (or dry)
    while (!dry) {
      int u;
      if (n_fetched < kStaticRounds) {
        u = wid + n_fetched * n_workers;
      } else {
        if (!have_dyn) {
          if (lane == 0) next_dyn = atomicAdd(&a.ctrl[0], 1u);
          have_dyn = true;
        }
        u = kStaticRounds * n_workers + (int)__shfl_sync(0xffffffffu, next_dyn, 0);
        have_dyn = false;
      }
      ++n_fetched;
      if (u >= total) { dry = true; break; }
      if (n_fetched >= kStaticRounds) {      // ask for the one after it now; the answer is used at the next call
        if (lane == 0) next_dyn = atomicAdd(&a.ctrl[0], 1u);
        have_dyn = true;
      }
      // at most kBufs earlier units still have stages in a buffer, so the record after the last kept one is free
      const int slot = n_kept % kUnitRing;
      decode_unit(a, sm, n_seg, u, &ring[slot], lane);
      __syncwarp();
      if (ring[slot].ok) { ++n_kept; iu = slot; is = 0; return; }
      if (ring[slot].sub == 0 && ring[slot].phase == 0 && lane == 0) atomicOr(a.err, ERR_BAD_ITEM);
    }
    iu = -1;
  };

  take_unit();
  while (true) {
    // issue while a buffer is free
    while (iu >= 0 && n_issued - n_done < kBufs) {
      const int b = n_issued % kBufs;
      const uint32_t buf = buf0 + b * kBufStride, bar = smem_u32(&sm.full[warp][b]);
      if (lane == 0) {
        sm.buf_unit[warp][b] = iu;
        sm.buf_stage[warp][b] = is;
        issue_stage(a, ring[iu], is, buf, bar, false);
        // the rows of this buffer may still be read by the bulk store of the stage that used it last
        bulk_wait_group_read0();
        issue_stage(a, ring[iu], is, buf, bar, true);
      }
      ++n_issued;
      if (++is == ring[iu].n_stages) take_unit();
    }
    if (n_done == n_issued) break;
    // consume the oldest stage
    const int b = n_done % kBufs;
    const uint32_t buf = buf0 + b * kBufStride, bar = smem_u32(&sm.full[warp][b]);
    __syncwarp();
    const int cu = sm.buf_unit[warp][b], cs = sm.buf_stage[warp][b];
    const UnitRec& r = ring[cu];
    if (!mbar_wait(bar, (uint32_t)(n_done / kBufs) & 1u)) {
      // the copies did not arrive: report, stop taking work, let what is in flight land (bounded again below)
      if (lane == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
      failed = true;
      iu = -1;
      dry = true;
      mbar_wait(bar, (uint32_t)(n_done / kBufs) & 1u);
      ++n_done;
      continue;
    }
    if (r.phase == 0) {
      if (cs == 0) {
#pragma unroll
        for (int jb = 0; jb < kImagePadMax / 16; ++jb)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[jb][e] = 0.f;
      }
      shrink_stage(a, r, cs, buf, acc, lane);
      if (cs == r.n_stages - 1 && !failed) shrink_finish(a, r, acc, sm.vsum[warp], lane);
    } else {
      bool ready = true;
      if (cs == 0 || cu_loaded != cu) {
        const uint32_t* state = a.job_state + 2 * (size_t)r.job;
        uint32_t spins = 0;
        while (ld_acquire(state) != kReady) {
          if (++spins >= kDepSpin) { ready = false; break; }
          __nanosleep(64);
        }
        if (ready) {
          const uint2* vf = a.vfrag + (size_t)r.job * (a.rp >> 4) * 32;
#pragma unroll
          for (int ks = 0; ks < kImagePadMax / 16; ++ks)
            vb[ks] = (ks < (r.rp >> 4)) ? __ldcg(vf + ks * 32 + lane) : make_uint2(0, 0);
          cu_loaded = cu;
        } else {
          if (lane == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
          failed = true;
          cu_loaded = -1;
        }
      }
      if (ready && cu_loaded == cu) expand_stage(a, r, cs, buf, vb, lane);
      if (cs == r.n_stages - 1 && !failed && lane == 0) {
        uint32_t* state = a.job_state + 2 * (size_t)r.job;
        const uint32_t old = atomicAdd(state + 1, 1u);
        if (old == (uint32_t)r.upj_e - 1) {      // every expand unit of the job has read v: reset for the next launch
          state[0] = 0;
          state[1] = 0;
        }
      }
    }
    __syncwarp();
    ++n_done;
  }
  // stores of y must have left shared memory before the CTA may go; the counter is reset by the last worker
  if (lane == 0) {
    bulk_wait_group0();
    __threadfence();        // a counter request that was never used must not pass the line below
    const uint32_t old = atomicAdd(&a.ctrl[1], 1u);
    if (old == (uint32_t)n_workers - 1) {
      a.ctrl[0] = 0;
      a.ctrl[1] = 0;
    }
  }
}

__host__ __device__ inline int stage_cols(int rp) {
  int c = (kStageBytes / (2 * rp)) & ~127;
  return c < 128 ? 128 : c;
}

}  // namespace

bool decode_stream_supported(const milora_ctx* ctx) {
  const milora_model_desc& d = ctx->desc;
  return d.dtype == MILORA_BF16 && d.d_model % 128 == 0 && d.d_ff % 128 == 0 && d.d_kv % 128 == 0 &&
         d.max_rank <= kImagePadMax;
}

// layers: host array, job_base not yet set.  n_seq_hint: sequences per layer (sizes the units).
milora_status launch_apply_decode_stream(milora_ctx* ctx, StreamLayer* layers, int n_layers, int n_seq_hint,
                                         cudaStream_t s) {
  if (!decode_stream_supported(ctx)) return MILORA_E_SHAPE;
  if (n_layers < 1) return MILORA_OK;
  StreamArgs a;
  std::memset(&a, 0, sizeof(a));
  a.err = ctx->d_err;
  a.rp = (ctx->desc.max_rank + 15) & ~15;
  a.cols = stage_cols(a.rp);
  double stages_per_job = 0;
  for (int m = 0; m < MILORA_NMOD; ++m) {
    module_dims(ctx->desc, m, &a.d1[m], &a.d2[m]);
    stages_per_job += ((a.d1[m] + a.cols - 1) / a.cols + (a.d2[m] + a.cols - 1) / a.cols) / (double)MILORA_NMOD;
  }
  const int workers = ctx->sm_count * kWarps;
  int us = ctx->stream_unit_stages;
  if (us < 1) {
    // enough units that every worker gets several; long units save partial sums and look-ups
    const double est = stages_per_job * std::max(1, n_seq_hint) * std::min(n_layers, kMaxStreamLayers);
    us = (int)(est / (workers * 4.0));
    us = std::max(1, std::min(us, 4));
  }
  a.unit_stages = us;
  int kcmax = 1;
  for (int m = 0; m < MILORA_NMOD; ++m)
    kcmax = std::max(kcmax, ((a.d1[m] + a.cols - 1) / a.cols + us - 1) / us);
  a.kcmax = kcmax;
  const size_t frag_bytes = (size_t)(a.rp >> 4) * 32 * sizeof(uint2);
  const size_t part_bytes = (size_t)kcmax * kR * a.rp * sizeof(float);
  // scratch of a launch: control words | job states | fragments | partial sums
  auto scratch_bytes = [&](size_t jobs) { return 256 + align256(jobs * 8) + align256(jobs * frag_bytes) + jobs * part_bytes; };
  const size_t cap_bytes = (size_t)512 << 20;
  const size_t smem = (size_t)kWarps * kBufs * kBufStride + sizeof(Smem);
  if (!ctx->stream_attr_set) {
    MILORA_CUDA(ctx, cudaFuncSetAttribute(decode_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ctx->stream_attr_set = true;
  }

  for (int l0 = 0; l0 < n_layers;) {
    // a launch takes as many layers as the record table and the scratch cap allow
    int l1 = l0;
    size_t jobs = 0;
    while (l1 < n_layers && l1 - l0 < kMaxStreamLayers) {
      const size_t j = (size_t)std::max(1, layers[l1].max_gather);
      if (l1 > l0 && scratch_bytes(jobs + j) > cap_bytes) break;
      layers[l1].job_base = (int32_t)jobs;
      jobs += j;
      ++l1;
    }
    const int n = l1 - l0;
    // The buffer is laid out for its capacity (jobs, bytes per job), not for the batch at hand, so a job's state
    // words never serve as anything else; every launch leaves them at zero, and they are cleared by the host only
    // when the buffer is new or after a launch that failed or timed out.
    if (jobs > ctx->stream_jobs_cap || frag_bytes > ctx->stream_frag_bytes || part_bytes > ctx->stream_part_bytes) {
      const size_t jc = std::max(jobs, ctx->stream_jobs_cap);
      const size_t fb = std::max(frag_bytes, ctx->stream_frag_bytes), pb = std::max(part_bytes, ctx->stream_part_bytes);
      const size_t need = 256 + align256(jc * 8) + align256(jc * fb) + jc * pb;
      MILORA_CUDA(ctx, cudaStreamSynchronize(s));
      if (ctx->d_stream) MILORA_CUDA(ctx, cudaFree(ctx->d_stream));
      ctx->d_stream = nullptr;
      ctx->stream_jobs_cap = 0;
      MILORA_CUDA(ctx, cudaMalloc(&ctx->d_stream, need));
      ctx->stream_jobs_cap = jc;
      ctx->stream_frag_bytes = fb;
      ctx->stream_part_bytes = pb;
      ctx->stream_dirty = true;
    }
    char* base = static_cast<char*>(ctx->d_stream);
    const size_t state_bytes = align256(ctx->stream_jobs_cap * 8);
    a.ctrl = reinterpret_cast<uint32_t*>(base);
    a.job_state = reinterpret_cast<uint32_t*>(base + 256);
    a.vfrag = reinterpret_cast<uint2*>(base + 256 + state_bytes);
    a.partial = reinterpret_cast<float*>(base + 256 + state_bytes + align256(ctx->stream_jobs_cap * ctx->stream_frag_bytes));
    if (ctx->stream_dirty) MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_stream, 0, 256 + state_bytes, s));
    a.n_layers = n;
    if (n == 1) {
      a.layers = nullptr;
      a.one = layers[l0];
    } else {
      // the records go through a pinned staging buffer, and only when they differ from what the device holds
      const size_t bytes = (size_t)n * sizeof(StreamLayer);
      if (!ctx->d_stream_layers) {
        MILORA_CUDA(ctx, cudaMalloc(&ctx->d_stream_layers, kMaxStreamLayers * sizeof(StreamLayer)));
        MILORA_CUDA(ctx, cudaHostAlloc(&ctx->h_stream_stage, 4 * kMaxStreamLayers * sizeof(StreamLayer), cudaHostAllocDefault));
        for (int i = 0; i < 4; ++i) MILORA_CUDA(ctx, cudaEventCreateWithFlags(&ctx->stream_stage_ev[i], cudaEventDisableTiming));
        ctx->stream_stage_next = 0;
        ctx->stream_layers_cached = 0;
      }
      StreamLayer* cached = static_cast<StreamLayer*>(ctx->h_stream_stage);     // slot of the last upload
      const int last = (ctx->stream_stage_next + 3) & 3;
      const bool same = ctx->stream_layers_cached == n &&
                        std::memcmp(cached + (size_t)last * kMaxStreamLayers, layers + l0, bytes) == 0;
      if (!same) {
        const int slot = ctx->stream_stage_next;
        MILORA_CUDA(ctx, cudaEventSynchronize(ctx->stream_stage_ev[slot]));    // its earlier copy has left the buffer
        StreamLayer* stage = cached + (size_t)slot * kMaxStreamLayers;
        std::memcpy(stage, layers + l0, bytes);
        MILORA_CUDA(ctx, cudaMemcpyAsync(ctx->d_stream_layers, stage, bytes, cudaMemcpyHostToDevice, s));
        MILORA_CUDA(ctx, cudaEventRecord(ctx->stream_stage_ev[slot], s));
        ctx->stream_stage_next = (slot + 1) & 3;
        ctx->stream_layers_cached = n;
      }
      a.layers = static_cast<const StreamLayer*>(ctx->d_stream_layers);
    }
    ctx->stream_dirty = true;       // stays set if the launch fails
    MILORA_CUDA(ctx, launch_pdl(decode_stream_kernel, dim3((unsigned)ctx->sm_count), dim3(kThreads), smem, s, a));
    ctx->stream_dirty = false;
    l0 = l1;
  }
  return MILORA_OK;
}

}  // namespace milora
