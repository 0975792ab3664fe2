// Decode path of Eq. 1 for bf16 on sm_100a as ONE persistent launch over any number of layers:
//   shrink:  v[job][t][j]  = s * gate_t * sum_c x[row_t][c] * A^T[j][c]
//   expand:  y[row_t][c]  += sum_j v[job][t][j] * B[j][c]
// for the gathered rows of the decode work lists (at most kGatherRows rows per job, all sharing one adapter;
// Section 3.3: the route is fixed per request, so the lists stay valid from step to step).
//
// Shape of the kernel
//   * One CTA per SM: W worker warps and one scheduler warp.  A worker owns kBufs shared-memory buffers and does
//     nothing but wait for a buffer to fill, contract it and hand it back.  Lane w of the scheduler warp is the
//     state machine of worker w: it takes units from the queue, reads their job records (two units ahead), and,
//     whenever one of the worker's buffers is free, writes the stage's descriptor and starts its copies (a "stage":
//     up to 8 KB of the A or B operand image as one contiguous cp.async.bulk, plus, for a shrink stage, the job's
//     rows of x, one bulk copy per row).  All bookkeeping of the ten workers thus costs one warp's instructions, and
//     none of its round trips to memory sits on a worker's path.
//   * Work is cut into units: `unit_stages` consecutive stages of one job's shrink or expand.  Units are numbered
//     so that every shrink unit of a job precedes all of its expand units, and the expand units of layer l come
//     after the shrink units of layer l + 1.  The first units are assigned by worker index, later ones come from a
//     counter (asked for ahead of time), so unequal units balance.
//   * A shrink unit leaves its partial x . A^T in global scratch and counts itself on the job; the unit that
//     arrives last adds the partials in unit order (deterministic), applies scale and gate, and publishes v as
//     ready-made mma.sync fragments (bf16 value + bf16 remainder, i.e. v to 2^-17).  Partial sums and fragments
//     travel as 8-byte {value, tag of this launch} pairs, so neither side needs a fence: an expand unit asks for
//     its job's fragments and repeats the request (bounded) until every tag is this launch's.  Units are handed out
//     in order and every worker is fed its units in order, so the unit with the smallest number that is not
//     finished can always proceed: no deadlock while all CTAs are resident (grid = number of SMs, one CTA per SM).
//   * Both contractions run on mma.sync m16n8k16 fed by ldmatrix from the operand images (the images are
//     8 x 16-byte core matrices, exactly what ldmatrix reads).  The path is bound by the adapter stream; the tensor
//     cores are used for the instruction count.
//     shrink: M = rank rows, N = rows of x, K = columns of d1.
//     expand: M = columns of d2, N = (row t, value | remainder), K = rank rows; the products are added to y with
//     red.global.add.noftz.bf16x2: y never travels to the SM, every element of y receives exactly one addition
//     (deterministic), and its error is half an ulp of y plus the bf16 rounding of the term (2^-9 of it).
//   * The job counters and the unit counter clean themselves up (the unit that adds a job up, the scheduler that
//     finishes last), so a launch leaves the scratch ready for the next one.
#include <algorithm>
#include <cstring>

#include "milora_internal.h"
#include "sm100_ptx.cuh"

namespace milora {
namespace {

using namespace ptx;

constexpr int kR = kGatherRows;
constexpr int kBufs = 2;                         // buffers (stages in flight) per worker
constexpr int kRowPad = 16;                      // keeps the rows of one stage on different banks
constexpr int kStaticRounds = 2;                 // units per worker assigned by index before the counter is used
constexpr int kMaxSeg = 2 * kMaxStreamLayers * MILORA_NMOD;
constexpr uint32_t kDepSpin = 1u << 22;          // repeats of a request for fragments or partial sums
constexpr uint32_t kSchedSpin = 1u << 26;        // rounds of the scheduler loop
constexpr int kMaxWarps = 10;

// Two shapes of the kernel: ten workers on 8 KB stages for the usual ranks (the warps hide each other's
// latencies; 20 stages in flight per SM), six on 16 KB stages for padded ranks of 48 and 64, whose smallest stage
// (one 128-column block of B) no longer fits 8 KB.
template <int WARPS, int STAGE>
struct Shape {
  static constexpr int kWarps = WARPS;           // workers; the scheduler is one more warp
  static constexpr int kStageBytes = STAGE;
  static constexpr int kSched = 2;               // scheduler warps; each serves half of the workers
  static constexpr int kThreads = (WARPS + kSched) * 32;
};
using ShapeSmall = Shape<10, 8192>;
using ShapeLarge = Shape<6, 16384>;

struct StreamArgs {
  int32_t* err;
  const StreamLayer* layers;   // device array, or nullptr: `one` is the only layer
  StreamLayer one;
  int n_layers;
  int d1[MILORA_NMOD], d2[MILORA_NMOD];
  int rp;                      // rank pad of the context: fixes the columns per stage
  int cols;                    // columns of d1 / d2 per stage
  int stage_bytes;             // adapter bytes per stage (the rows of x follow them in a buffer)
  int buf_stride;              // bytes from one buffer to the next: stage + kR rows of x, rounded up
  int unit_stages;             // stages per unit
  int kcmax;                   // most shrink units per job over the modules
  uint32_t* ctrl;              // [0] units handed out beyond the static rounds, [1] schedulers that have finished
  uint32_t* job_state;         // [jobs]: shrink units of the job that have delivered their partial sums
  uint32_t epoch;              // tag of this launch (never 0): marks the values written by it
  uint2* partial;              // [jobs][kcmax][kR][rp] of {value, epoch}
  uint4* vfrag;                // [jobs][rp / 16][32] of {word 0, epoch, word 1, epoch}
};

// What a worker needs to know about its work.  The scheduler writes a unit's record when it takes the unit and
// two words per stage before it starts the stage's copies; the worker reads both after the buffer's barrier has
// completed (the scheduler's arrive on that barrier releases them).  A worker has at most kBufs + 1 units alive
// (one per buffer, one being issued), so kUnitRing records take turns.
enum StageKind { STAGE_SHRINK = 0, STAGE_EXPAND = 1, STAGE_STOP = 2 };
constexpr int kUnitRing = 4;
struct UnitRec {
  char* y_base;                // expand: first element of the module's Y
  int32_t rows[kR];            // expand: rows of y
  float w[kR];                 // shrink: scale * gate of each row of the job (used when the unit ends)
  int32_t n, jb, d;            // rows of the job, rank blocks of 16, row length of y
  int32_t job, sub, upj_s;
};
struct StageWord {             // ncols | slot << 16 | first << 20 | last << 21 | kind << 22, then the first column
  uint32_t bits;
  int32_t c0;
};
__host__ __device__ inline uint32_t stage_bits(int ncols, int slot, bool first, bool last, int kind) {
  return (uint32_t)ncols | (uint32_t)slot << 16 | (uint32_t)first << 20 | (uint32_t)last << 21 | (uint32_t)kind << 22;
}

struct Smem {
  StreamLayer layers[kMaxStreamLayers];
  int32_t seg_base[kMaxSeg + 1];
  int32_t first[kMaxStreamLayers][MILORA_NMOD + 1];
  int32_t upj[2][MILORA_NMOD];
  UnitRec unit[kMaxWarps][kUnitRing];
  StageWord stage[kMaxWarps][kBufs];
  uint64_t full[kMaxWarps][kBufs], empty[kMaxWarps][kBufs];
  uint4 rec[kMaxWarps][3][4];         // job records of the units a scheduler lane has located (cp.async targets)
  volatile int32_t hint[kMaxWarps];   // job of the expand unit taken last for each worker (-1: none): what to ask fragments for
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
// Two neighbouring elements of y += (v0, v1) in bf16, performed by the L2 (one rounding of each sum).  The packed
// form is a native operation; the scalar bf16 form is not (measured: 40 us for one row of 4096 columns).
__device__ __forceinline__ void red_add_bf16x2(void* addr, float v0, float v1) {
  const uint32_t h = pack_bf16(v0, v1);
  asm volatile("red.global.add.noftz.bf16x2 [%0], %1;" ::"l"(addr), "r"(h) : "memory");
}
// A value that travels together with the tag of the launch that wrote it, as one 8-byte access (8-byte accesses
// are single-copy atomic): whoever reads the right tag has the right value, without a flag or a fence.
__device__ __forceinline__ void st_tagged1(uint2* p, uint32_t w, uint32_t tag) {
  asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(w), "r"(tag) : "memory");
}
__device__ __forceinline__ uint2 ld_tagged1(const uint2* p) {
  uint2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
// A fragment word travels together with the tag of the launch that wrote it, as one 8-byte access (8-byte
// accesses are single-copy atomic): whoever reads the right tag has the right word, without a flag or a fence.
__device__ __forceinline__ void st_tagged(uint4* p, uint32_t w0, uint32_t w1, uint32_t tag) {
  asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(w0), "r"(tag) : "memory");
  asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(reinterpret_cast<char*>(p) + 8), "r"(w1), "r"(tag) : "memory");
}
__device__ __forceinline__ uint4 ld_tagged(const uint4* p) {
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.z), "=r"(v.w) : "l"(reinterpret_cast<const char*>(p) + 8) : "memory");
  return v;
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

// ---- scheduler: one lane per worker -------------------------------------------------------------------------
// A unit that has been found in the work lists and whose 64-byte job record is on its way to shared memory
// (cp.async: the lane holds no register for it and never waits when it asks).
struct UnitLoc {
  int li, phase, m, job_local, sub, slot;      // slot: which of the lane's three record buffers the record goes to
  bool valid;
};
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// `seg` is the lane's cursor into the prefix table: unit numbers only grow, so the search starts where the last
// one ended.
__device__ __forceinline__ void locate_unit(const StreamArgs& a, Smem& sm, int n_seg, int u, int w, int slot, int* seg,
                                            UnitLoc* x) {
  int sg = *seg;
  if (sg + 8 < n_seg && sm.seg_base[sg + 8] <= u) {
    // far ahead (a lane's first units): last segment whose base is <= u, by bisection
    int lo = sg + 8, hi = n_seg - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sm.seg_base[mid] <= u) lo = mid; else hi = mid - 1;
    }
    sg = lo;
  }
  while (sg + 1 < n_seg && sm.seg_base[sg + 1] <= u) ++sg;
  *seg = sg;
  const int p = sg / MILORA_NMOD;
  x->m = sg - p * MILORA_NMOD;
  pos_to_layer(p, a.n_layers, &x->li, &x->phase);
  const int local = u - sm.seg_base[sg];
  const int upj = sm.upj[x->phase][x->m];
  // local / upj for small non-negative numbers: the float quotient of (local + 0.5) is never close to an integer
  const int jq = __float2int_rz(__fdividef((float)local + 0.5f, (float)upj));
  x->job_local = sm.first[x->li][x->m] + jq;
  x->sub = local - jq * upj;
  const StreamLayer& L = sm.layers[x->li];
  const uint4* jp = reinterpret_cast<const uint4*>(L.ws + L.off_gather) + (size_t)x->job_local * (kJobInts / 4);
  const uint32_t dst = smem_u32(&sm.rec[w][slot][0]);
#pragma unroll
  for (int i = 0; i < 4; ++i) cp_async16(dst + 16 * i, jp + i);
  cp_async_commit();
  x->slot = slot;
  x->valid = true;
}

// A unit as the scheduler lane keeps it while it issues the unit's stages.
struct Unit {
  const char* img;             // operand image of the phase, at the unit's first stage
  const char* x0;              // shrink: X of the module at the unit's first column
  int32_t rows[kR];
  int32_t n, rp, d, phase, c_begin, n_stages, slot;
};
// Checks the job record (a damaged one is skipped by its shrink and its expand units alike), derives the unit and
// writes its record for the worker.
__device__ __forceinline__ bool decode_unit(const StreamArgs& a, const Smem& sm, const UnitLoc& x, const uint4* piece,
                                            Unit* un, UnitRec* rec) {
  const StreamLayer& L = sm.layers[x.li];
  const int m = x.m;
  const uint4 p0 = piece[0], p1 = piece[1], p2 = piece[2], p3 = piece[3];
  const char* At = reinterpret_cast<const char*>(((uint64_t)p0.y << 32) | p0.x);
  const int rank = (int)p1.x, count = (int)p1.w;
  const float scale = __uint_as_float(p1.y);
  const int rows[kR] = {(int)p2.x, (int)p2.y, (int)p2.z, (int)p2.w};
  const float gate[kR] = {__uint_as_float(p3.x), __uint_as_float(p3.y), __uint_as_float(p3.z), __uint_as_float(p3.w)};
  const int rpj = (rank + 15) & ~15;
  bool ok = rank > 0 && rpj <= a.rp && count > 0 && count <= kR && At != nullptr && (int)p1.z == m &&
            L.X[m] != nullptr && L.Y[m] != nullptr;
#pragma unroll
  for (int t = 0; t < kR; ++t)
    if (t < count && (rows[t] < 0 || rows[t] >= L.T)) ok = false;
  if (!ok) return false;
  const int d1 = a.d1[m], d2 = a.d2[m];
  const int d = x.phase ? d2 : d1;
  const int stages = (d + a.cols - 1) / a.cols;
  const AdapterLayout al = adapter_layout(d1, d2, rank, 2);
  const size_t off = x.phase ? al.off_b_img : al.off_a_img;
  un->c_begin = x.sub * a.unit_stages * a.cols;
  // both images are contiguous in column order: rp * 2 bytes per column
  un->img = At + off + (size_t)un->c_begin * rpj * 2;
  un->x0 = static_cast<const char*>(L.X[m]) + (size_t)un->c_begin * 2;
#pragma unroll
  for (int t = 0; t < kR; ++t) un->rows[t] = rows[t];
  un->n = count; un->rp = rpj; un->d = d; un->phase = x.phase;
  un->n_stages = min(a.unit_stages, stages - x.sub * a.unit_stages);
  rec->y_base = static_cast<char*>(L.Y[m]);
#pragma unroll
  for (int t = 0; t < kR; ++t) {
    rec->rows[t] = rows[t];
    rec->w[t] = t < count ? scale * gate[t] : 0.f;
  }
  rec->n = count; rec->jb = rpj >> 4; rec->d = d;
  rec->job = L.job_base + x.job_local; rec->sub = x.sub; rec->upj_s = sm.upj[0][m];
  return true;
}

// Stage `is` of the unit into a free buffer of the worker: its two words, then its copies.
__device__ __forceinline__ void issue_stage(const StreamArgs& a, const Unit& un, int is, StageWord* sw, uint32_t buf,
                                            uint32_t bar) {
  const int c_off = is * a.cols;                       // columns from the unit's first one
  const int ncols = min(a.cols, un.d - un.c_begin - c_off);
  sw->bits = stage_bits(ncols, un.slot, is == 0, is == un.n_stages - 1, un.phase);
  sw->c0 = un.c_begin + c_off;
  const uint32_t bytes_img = (uint32_t)ncols * un.rp * 2, bytes_row = (uint32_t)ncols * 2;
  const int n_rows = un.phase == 0 ? un.n : 0;
  // the arrive releases the words and the unit's record to the worker, whose wait on the barrier acquires them
  mbar_expect_tx(bar, bytes_img + (uint32_t)n_rows * bytes_row);
  // the operand images are read once per launch: evict first, so that what the launch reads again (partial sums,
  // fragments, job records, the rows of y it adds to) keeps its place in L2
  bulk_g2s_hint(buf, un.img + (size_t)c_off * un.rp * 2, bytes_img, bar, l2_evict_first_policy());
  const uint32_t rstride = (uint32_t)a.cols * 2 + kRowPad;
  for (int t = 0; t < n_rows; ++t)
    bulk_g2s(buf + a.stage_bytes + t * rstride, un.x0 + ((size_t)un.rows[t] * un.d + c_off) * 2, bytes_row, bar);
}

// ---- worker: shrink -------------------------------------------------------------------------------------------
// One stage into the unit's accumulators.  JB = rank blocks of 16.  The instructions of one 64-column chunk are
// grouped by kind (x fragments, ldmatrix, MMA) so that independent ones follow each other: the asm statements keep
// their order, and a chain ldmatrix -> mma -> next ldmatrix would run at one latency per step.  Consecutive k steps
// go to independent accumulator sets, which are added when the unit ends.
// acc[s * JB + jb] is a 16 x 8 tile (rank rows jb*16.., rows of x): c0, c1 = (rank row g, x rows 2q, 2q+1),
// c2, c3 = (rank row g + 8, same x rows).
constexpr int kAccSets = 8;     // accumulator tiles a worker holds: steps-per-batch x JB
template <int JB>
__device__ __forceinline__ void shrink_stage(const StreamArgs& a, int n, int ncols, uint32_t buf, float (&acc)[kAccSets][4],
                                             int lane) {
  constexpr int SB = JB <= 2 ? 4 : 2;          // k steps whose loads are issued together
  const int g = lane >> 2, q = lane & 3, mi = lane >> 3;
  constexpr int rp = JB * 16;
  const uint32_t rstride = (uint32_t)a.cols * 2 + kRowPad;
  const bool x_ok = g < n;
  const uint32_t xrow = buf + a.stage_bytes + (x_ok ? g : 0) * rstride + 4 * q;
  // ldmatrix row address of this lane inside a 64-column chunk, for k step 0 and rank block 0:
  // core matrix (j / 8, k / 8) at ((k / 8) * (rp / 8) + j / 8) * 128
  const uint32_t lane_off = (uint32_t)(((mi >> 1) * (rp >> 3) + (mi & 1)) * 128 + (lane & 7) * 16);
  for (int kc = 0; kc < (ncols >> 6); ++kc) {
    const uint32_t chunk = buf + (uint32_t)kc * rp * 128 + lane_off;
#pragma unroll
    for (int s0 = 0; s0 < 4; s0 += SB) {
      uint32_t b0[SB], b1[SB], am[SB][JB][4];
#pragma unroll
      for (int s = 0; s < SB; ++s) {
        b0[s] = b1[s] = 0;
        if (x_ok) {
          b0[s] = lds32(xrow + (kc * 64 + (s0 + s) * 16) * 2);
          b1[s] = lds32(xrow + (kc * 64 + (s0 + s) * 16 + 8) * 2);
        }
      }
#pragma unroll
      for (int s = 0; s < SB; ++s)
#pragma unroll
        for (int jb = 0; jb < JB; ++jb)
          ldmatrix_x4(chunk + (uint32_t)((2 * (s0 + s)) * (rp >> 3) + 2 * jb) * 128, am[s][jb][0], am[s][jb][1], am[s][jb][2],
                      am[s][jb][3]);
#pragma unroll
      for (int s = 0; s < SB; ++s)
#pragma unroll
        for (int jb = 0; jb < JB; ++jb)
          mma_16816(acc[s * JB + jb], am[s][jb][0], am[s][jb][1], am[s][jb][2], am[s][jb][3], b0[s], b1[s]);
    }
  }
}

// End of a shrink unit, first half: partial products to scratch and one count on the job.  The answer of the count
// (lane 0) is not looked at here: the worker goes on with its next stage and calls shrink_finalize afterwards, so
// the round trip of the atomic is not on its path.
struct PendingCount {
  uint32_t old;          // lane 0: units of the job that had arrived before this one
  int32_t job, upj_s, jb;
  float w;               // scale * gate of this lane's row of v (row t = lane / 8), 0 beyond the job's rows
  bool valid;
};
template <int JB>
__device__ __forceinline__ void shrink_publish(const StreamArgs& a, const UnitRec& dsc, float (&acc)[kAccSets][4],
                                               PendingCount* pc, int lane) {
  constexpr int SB = JB <= 2 ? 4 : 2;
  const int g = lane >> 2, q = lane & 3;
  const int job = dsc.job;
  uint2* part = a.partial + ((size_t)job * a.kcmax + dsc.sub) * kR * a.rp;
  if (q < 2) {
#pragma unroll
    for (int jb = 0; jb < JB; ++jb) {
      float c[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        c[e] = acc[jb][e];
#pragma unroll
        for (int s = 1; s < SB; ++s) c[e] += acc[s * JB + jb][e];      // fixed order: set 0, 1, ...
      }
      const int j = jb * 16 + g;
      st_tagged1(part + (2 * q) * a.rp + j, __float_as_uint(c[0]), a.epoch);
      st_tagged1(part + (2 * q + 1) * a.rp + j, __float_as_uint(c[1]), a.epoch);
      st_tagged1(part + (2 * q) * a.rp + j + 8, __float_as_uint(c[2]), a.epoch);
      st_tagged1(part + (2 * q + 1) * a.rp + j + 8, __float_as_uint(c[3]), a.epoch);
    }
  }
  pc->job = job; pc->upj_s = dsc.upj_s; pc->jb = JB;
  pc->w = dsc.w[g >> 1];
  pc->valid = true;
  pc->old = 0;
  // The count only decides who adds the job up; the partial sums carry this launch's tag, so no fence is needed
  // (a fence here would wait for every addition into y that this warp still has under way).
  if (lane == 0) pc->old = atomicAdd(a.job_state + job, 1u);
}

// Second half: the unit that arrived last adds the job's partial sums in unit order and publishes v as the
// fragments of the expand MMAs' second operand (K = rank rows, N = 8): column n = g holds row t = g / 2 of v, as its
// bf16 value for even g and as the remainder after that rounding for odd g.  Each lane computes the values of its
// own fragment.  A partial sum whose tag is not this launch's yet (its store is still on the way) is asked for
// again, a bounded number of times.  The job's counter goes back to zero for the next launch.
// Returns false when a partial sum never arrived.
__device__ __forceinline__ bool shrink_finalize(const StreamArgs& a, PendingCount* pc, int lane) {
  if (!pc->valid) return true;
  pc->valid = false;
  const uint32_t old = __shfl_sync(0xffffffffu, pc->old, 0);
  if (old != (uint32_t)pc->upj_s - 1) return true;
  const int g = lane >> 2, q = lane & 3;
  const int t = g >> 1;
  const bool rem = g & 1;
  const uint2* base = a.partial + (size_t)pc->job * a.kcmax * kR * a.rp + t * a.rp;
  const size_t ustride = (size_t)kR * a.rp;
  uint4* out = a.vfrag + (size_t)pc->job * (a.rp >> 4) * 32;
  if (lane == 0) a.job_state[pc->job] = 0;
  bool all_ok = true;
  for (int ks = 0; ks < pc->jb; ++ks) {
    const uint2* vp = base + ks * 16 + 2 * q;
    float v4[4] = {0.f, 0.f, 0.f, 0.f};
    for (int c0 = 0; c0 < pc->upj_s; c0 += 4) {
      uint2 p[4][4];
      uint32_t spins = 0;
      while (true) {
        bool ok = true;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint2* u = vp + (size_t)min(c0 + i, pc->upj_s - 1) * ustride;
          p[i][0] = ld_tagged1(u);
          p[i][1] = ld_tagged1(u + 1);
          p[i][2] = ld_tagged1(u + 8);
          p[i][3] = ld_tagged1(u + 9);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) ok = ok && p[i][e].y == a.epoch;
        if (__all_sync(0xffffffffu, ok)) break;
        if (++spins >= kDepSpin) { all_ok = false; break; }
        __nanosleep(100);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (c0 + i < pc->upj_s) {
#pragma unroll
          for (int e = 0; e < 4; ++e) v4[e] += __uint_as_float(p[i][e].x);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) v4[i] *= pc->w;
    uint32_t w0 = pack_bf16(v4[0], v4[1]), w1 = pack_bf16(v4[2], v4[3]);
    if (rem) {
      const uint32_t h0 = w0, h1 = w1;
      w0 = pack_bf16(v4[0] - bf16_lo(h0), v4[1] - bf16_hi(h0));
      w1 = pack_bf16(v4[2] - bf16_lo(h1), v4[3] - bf16_hi(h1));
    }
    if (all_ok) st_tagged(out + ks * 32 + lane, w0, w1, a.epoch);
  }
  return all_ok;
}

// ---- worker: expand -------------------------------------------------------------------------------------------
// One stage, added to y in global memory.  KS = rank blocks of 16.  NS steps of 16 columns are handled together,
// again grouped by kind of instruction.
template <int KS>
__device__ __forceinline__ void expand_stage(const UnitRec& dsc, int ncols, int c0, uint32_t buf,
                                             const uint2 (&vb)[kImagePadMax / 16], int lane) {
  constexpr int NS = KS <= 2 ? 8 / KS : 2;
  constexpr int rp = KS * 16;
  const int g = lane >> 2, q = lane & 3, mi = lane >> 3;
  const bool row_ok = q < dsc.n;
  // ldmatrix takes any eight rows for a matrix: the first M half of a step is given the step's even columns and
  // the second half the odd ones, so that the accumulators of this lane are columns 2g and 2g + 1 of row t = q:
  // two neighbouring elements of y, which one packed addition updates.
  __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(dsc.y_base) + (size_t)(row_ok ? dsc.rows[q] : 0) * dsc.d + c0 + 2 * g;
  // row address inside a 128-column block for rank step 0, column step 0: column n of the block sits in
  // core matrix (n / 8, k / 8) at ((k / 8) * 16 + n / 8) * 128, row n % 8
  const int n_loc = 2 * (lane & 7) + (mi & 1);
  const uint32_t lane_off = (uint32_t)(((mi >> 1) * 16 + (n_loc >> 3)) * 128 + (n_loc & 7) * 16);
  for (int nb = 0; nb < (ncols >> 7); ++nb) {
    const uint32_t blk = buf + (uint32_t)nb * rp * 256 + lane_off;
#pragma unroll
    for (int n0 = 0; n0 < 8; n0 += NS) {
      uint32_t am[NS][KS][4];
      float c[NS][4];
#pragma unroll
      for (int ns = 0; ns < NS; ++ns)
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          ldmatrix_x4(blk + (uint32_t)((2 * ks) * 16 + 2 * (n0 + ns)) * 128, am[ns][ks][0], am[ns][ks][1], am[ns][ks][2],
                      am[ns][ks][3]);
#pragma unroll
      for (int ns = 0; ns < NS; ++ns) {
        c[ns][0] = c[ns][1] = c[ns][2] = c[ns][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          mma_16816(c[ns], am[ns][ks][0], am[ns][ks][1], am[ns][ks][2], am[ns][ks][3], vb[ks].x, vb[ks].y);
      }
      // c0 + c1: column 2g of the step, row t = q (value part + remainder part); c2 + c3: column 2g + 1
      if (row_ok) {
#pragma unroll
        for (int ns = 0; ns < NS; ++ns)
          red_add_bf16x2(yp + nb * 128 + (n0 + ns) * 16, c[ns][0] + c[ns][1], c[ns][2] + c[ns][3]);
      }
    }
  }
}

// ---- the kernel --------------------------------------------------------------------------------------------
template <class SH>
__global__ void __launch_bounds__(SH::kThreads, 1) decode_stream_kernel(StreamArgs a) {
  constexpr int kWarps = SH::kWarps;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw + (size_t)kWarps * kBufs * a.buf_stride);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int w = 0; w < kWarps; ++w) {
      for (int b = 0; b < kBufs; ++b) {
        mbar_init(smem_u32(&sm.full[w][b]), 1);
        mbar_init(smem_u32(&sm.empty[w][b]), 1);
      }
      sm.hint[w] = -1;
    }
    fence_barrier_init();
  }
  pdl_launch_dependents();
  __syncthreads();
  pdl_wait();

  // Layer records and the first job of every (layer, module): every thread of the CTA takes a share, so that the
  // look-ups of a 32-layer call (two dependent loads each) run side by side instead of one warp's eight rounds.
  {
    const int L = a.n_layers;
    const uint4* src = reinterpret_cast<const uint4*>(a.layers);
    uint4* dst = reinterpret_cast<uint4*>(sm.layers);
    if (a.layers) {
      for (int i = tid; i < L * (int)(sizeof(StreamLayer) / 16); i += SH::kThreads) dst[i] = src[i];
    } else if (tid == 0) {
      sm.layers[0] = a.one;
    }
    if (tid < MILORA_NMOD) {
      const int ss = (a.d1[tid] + a.cols - 1) / a.cols, se = (a.d2[tid] + a.cols - 1) / a.cols;
      sm.upj[0][tid] = (ss + a.unit_stages - 1) / a.unit_stages;
      sm.upj[1][tid] = (se + a.unit_stages - 1) / a.unit_stages;
    }
    __syncthreads();
    for (int i = tid; i < L * (MILORA_NMOD + 1); i += SH::kThreads) {
      const int li = i / (MILORA_NMOD + 1), m = i % (MILORA_NMOD + 1);
      const StreamLayer& Ly = sm.layers[li];
      const int n_jobs = max(0, min(Ly.ws[Ly.off_header + H_NGATHER], Ly.max_gather));
      sm.first[li][m] = max(0, min(Ly.ws[Ly.off_mod_gather + m], n_jobs));
    }
    __syncthreads();
    // unit counts per (queue position, module), left where their prefix sums will stand
    for (int i = tid; i < 2 * L * MILORA_NMOD; i += SH::kThreads) {
      const int p = i / MILORA_NMOD, m = i % MILORA_NMOD;
      int li, phase;
      pos_to_layer(p, L, &li, &phase);
      const StreamLayer& Ly = sm.layers[li];
      int v = max(0, sm.first[li][m + 1] - sm.first[li][m]) * sm.upj[phase][m];
      if (Ly.X[m] == nullptr || Ly.Y[m] == nullptr) v = 0;
      sm.seg_base[i + 1] = v;
    }
    __syncthreads();
  }

  if (warp >= kWarps) {
    // ================= scheduler =================
    const int sched = warp - kWarps;
    constexpr int kPerSched = (kWarps + SH::kSched - 1) / SH::kSched;
    const int L = a.n_layers;
    const int n_seg = 2 * L * MILORA_NMOD;
    if (sched == 0) {
    {
      // prefix sums of the unit counts, 32 entries per pass
      int carry = 0;
      if (lane == 0) sm.seg_base[0] = 0;
      for (int b = 0; b < n_seg; b += 32) {
        const int i = b + lane;
        int v = i < n_seg ? sm.seg_base[i + 1] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, v, o);
          if (lane >= o) v += t;
        }
        if (i < n_seg) sm.seg_base[i + 1] = carry + v;
        carry += __shfl_sync(0xffffffffu, v, 31);
      }
    }
    __syncwarp();
    }
    // the other scheduler warps wait for the table
    named_barrier(1, SH::kSched * 32);
    const int total = sm.seg_base[n_seg];

    bool timed_out = false;
    if (lane < kPerSched && sched * kPerSched + lane < kWarps) {
      const int w = sched * kPerSched + lane;
      const int n_workers = (int)gridDim.x * kWarps;
      const int wid = w * (int)gridDim.x + (int)blockIdx.x;     // neighbouring units go to different SMs
      const uint32_t buf0 = smem_u32(smem_raw) + (uint32_t)(w * kBufs) * a.buf_stride;
      int n_fetched = 0, n_located = 0, n_issued = 0, n_kept = 0, is = 0, seg = 0;
      bool dry = false, have_cur = false, stop_sent = false;
      // How far a lane looks ahead decides what the workers still hold when the queue runs dry, i.e. how long the
      // last of them works alone.  Short units (one or two stages, 2 to 4 us) need the full depth to hide the
      // counter's and the record's round trips: two located units and one claimed number.  Long units give the
      // lane time: one located unit, and the counter is asked when the number is needed.
      const bool deep = a.unit_stages <= 2;
      uint32_t next_dyn = deep ? atomicAdd(&a.ctrl[0], 1u) : 0u;     // used by the third look-ahead; the answer has time to come
      UnitLoc q0, q1;
      Unit cur;
      auto fetch_q1 = [&]() {
        q1.valid = false;
        if (dry) return;
        int u;
        if (n_fetched < kStaticRounds) {
          u = wid + n_fetched * n_workers;
        } else {
          if (deep) {
            u = kStaticRounds * n_workers + (int)next_dyn;
            next_dyn = atomicAdd(&a.ctrl[0], 1u);        // for the call after this one
          } else {
            u = kStaticRounds * n_workers + (int)atomicAdd(&a.ctrl[0], 1u);
          }
        }
        ++n_fetched;
        if (u >= total) { dry = true; return; }
        locate_unit(a, sm, n_seg, u, w, n_located % 3, &seg, &q1);
        ++n_located;
      };
      fetch_q1();
      q0 = q1;
      if (deep) fetch_q1(); else q1.valid = false;
      uint32_t round = 0;
      for (; round < kSchedSpin && !stop_sent; ++round) {
        if (!have_cur && q0.valid) {
          // at most kBufs earlier units still have stages in a buffer, so the record after the last kept one is free
          const int slot = n_kept % kUnitRing;
          // the record of q0 was asked for before that of q1: all but the newest request must have landed
          if (q1.valid) cp_async_wait<1>(); else cp_async_wait<0>();
          const bool ok = decode_unit(a, sm, q0, sm.rec[w][q0.slot], &cur, &sm.unit[w][slot]);
          if (!ok && q0.sub == 0 && q0.phase == 0) atomicOr(a.err, ERR_BAD_ITEM);
          if (deep) {
            q0 = q1;
            fetch_q1();
          } else {
            fetch_q1();
            q0 = q1;
            q1.valid = false;
          }
          if (ok) {
            have_cur = true;
            is = 0;
            cur.slot = slot;
            ++n_kept;
            if (cur.phase == 1) sm.hint[w] = sm.unit[w][slot].job;
          }
        }
        // stages of the current unit into every free buffer, or, when nothing is left, the word that ends the worker
        bool progress = false;
#pragma unroll
        for (int rep = 0; rep < kBufs; ++rep) {
          if (!(have_cur || (!q0.valid && !stop_sent))) break;
          const int b = n_issued % kBufs, k = n_issued / kBufs;
          if (k > 0 && !mbar_test_wait(smem_u32(&sm.empty[w][b]), (uint32_t)(k - 1) & 1u)) break;
          const uint32_t bar = smem_u32(&sm.full[w][b]);
          if (have_cur) {
            issue_stage(a, cur, is, &sm.stage[w][b], buf0 + b * a.buf_stride, bar);
            if (++is == cur.n_stages) have_cur = false;
          } else {
            sm.stage[w][b].bits = stage_bits(0, 0, false, false, STAGE_STOP);
            mbar_arrive(bar);
            stop_sent = true;
          }
          ++n_issued;
          progress = true;
        }
        if (!progress && have_cur) __nanosleep(32);
      }
      timed_out = !stop_sent;
      __threadfence();        // a counter request that was never used must not pass the count of finished CTAs
    }
    if (__any_sync(0xffffffffu, timed_out) && lane == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
    __syncwarp();
    // the unit counter is reset by the scheduler that finishes last
    if (lane == 0) {
      const uint32_t old = atomicAdd(&a.ctrl[1], 1u);
      if (old == gridDim.x * SH::kSched - 1) {
        a.ctrl[0] = 0;
        a.ctrl[1] = 0;
      }
    }
    return;
  }

  // ================= worker =================
  const uint32_t buf0 = smem_u32(smem_raw) + (uint32_t)(warp * kBufs) * a.buf_stride;
  float acc[kAccSets][4];
  PendingCount pend;
  pend.valid = false;
  uint4 vb_pf[kImagePadMax / 16];      // fragments asked for ahead of time, and the job they belong to
  int pf_job = -1;
  uint2 vb[kImagePadMax / 16];
  bool failed = false;
  const int ks_ctx = a.rp >> 4;
  for (int n_done = 0;; ++n_done) {
    const int b = n_done % kBufs;
    const uint32_t buf = buf0 + b * a.buf_stride;
    // the scheduler says which job's expand unit comes next: ask for its fragments while waiting
    {
      const int hj = sm.hint[warp];
      if (hj >= 0 && hj != pf_job) {
        const uint4* vf = a.vfrag + (size_t)hj * ks_ctx * 32;
#pragma unroll
        for (int ks = 0; ks < kImagePadMax / 16; ++ks)
          if (ks < ks_ctx) vb_pf[ks] = ld_tagged(vf + ks * 32 + lane);
        pf_job = hj;
      }
    }
    if (!mbar_wait(smem_u32(&sm.full[warp][b]), (uint32_t)(n_done / kBufs) & 1u)) {
      // nothing arrived within the limit: report and leave (the scheduler gives up on its own limit; copies that
      // were started have had the same time to land)
      failed = true;
      break;
    }
    const uint32_t bits = sm.stage[warp][b].bits;
    const int kind = (int)(bits >> 22);
    if (kind == STAGE_STOP) break;
    const int ncols = (int)(bits & 0xFFFFu), c0 = sm.stage[warp][b].c0;
    const bool first = (bits >> 20) & 1u, last = (bits >> 21) & 1u;
    const UnitRec& dsc = sm.unit[warp][(bits >> 16) & 15u];
    const int jb = dsc.jb;
    if (kind == STAGE_SHRINK) {
      if (first) {
#pragma unroll
        for (int i = 0; i < kAccSets; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
      }
      const int n = dsc.n;
      switch (jb) {
        case 1: shrink_stage<1>(a, n, ncols, buf, acc, lane); break;
        case 2: shrink_stage<2>(a, n, ncols, buf, acc, lane); break;
        case 3: shrink_stage<3>(a, n, ncols, buf, acc, lane); break;
        default: shrink_stage<4>(a, n, ncols, buf, acc, lane); break;
      }
      if (!shrink_finalize(a, &pend, lane)) failed = true;      // the count of the unit before this one has had time to answer
      if (last) {
        switch (jb) {
          case 1: shrink_publish<1>(a, dsc, acc, &pend, lane); break;
          case 2: shrink_publish<2>(a, dsc, acc, &pend, lane); break;
          case 3: shrink_publish<3>(a, dsc, acc, &pend, lane); break;
          default: shrink_publish<4>(a, dsc, acc, &pend, lane); break;
        }
      }
    } else {
      bool have = true;
      if (first) {
        // fragments of v: those asked for ahead of time when they are this job's, asked for again until every tag
        // is this launch's (the job's shrink units may not all have finished; the last of them may even be the
        // count this very warp has not looked at yet)
        const int job = dsc.job;
        const uint4* vf = a.vfrag + (size_t)job * ks_ctx * 32;
        uint4 f[kImagePadMax / 16];
#pragma unroll
        for (int ks = 0; ks < kImagePadMax / 16; ++ks) {
          f[ks] = make_uint4(0, a.epoch, 0, a.epoch);
          if (ks < jb) f[ks] = (pf_job == job) ? vb_pf[ks] : ld_tagged(vf + ks * 32 + lane);
        }
        uint32_t spins = 0;
        while (true) {
          bool mine = true;
#pragma unroll
          for (int ks = 0; ks < kImagePadMax / 16; ++ks) mine = mine && f[ks].y == a.epoch && f[ks].w == a.epoch;
          if (__all_sync(0xffffffffu, mine)) break;
          if (++spins >= kDepSpin) { have = false; break; }
          if (!shrink_finalize(a, &pend, lane)) failed = true;
          __nanosleep(100);
#pragma unroll
          for (int ks = 0; ks < kImagePadMax / 16; ++ks)
            if (ks < jb) f[ks] = ld_tagged(vf + ks * 32 + lane);
        }
#pragma unroll
        for (int ks = 0; ks < kImagePadMax / 16; ++ks) vb[ks] = make_uint2(f[ks].x, f[ks].z);
        if (!have) {
          failed = true;
#pragma unroll
          for (int ks = 0; ks < kImagePadMax / 16; ++ks) vb[ks] = make_uint2(0, 0);     // the unit adds nothing
        }
      }
      switch (jb) {
        case 1: expand_stage<1>(dsc, ncols, c0, buf, vb, lane); break;
        case 2: expand_stage<2>(dsc, ncols, c0, buf, vb, lane); break;
        case 3: expand_stage<3>(dsc, ncols, c0, buf, vb, lane); break;
        default: expand_stage<4>(dsc, ncols, c0, buf, vb, lane); break;
      }
      if (!shrink_finalize(a, &pend, lane)) failed = true;
    }
    // every lane's reads of the buffer and of the descriptor are done (the MMAs needed them): hand it back
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&sm.empty[warp][b]));
  }
  if (!shrink_finalize(a, &pend, lane)) failed = true;
  if (failed && lane == 0) atomicOr(a.err, ERR_WAIT_TIMEOUT);
}

// Columns of d1 / d2 per stage: as many 128-column blocks as the stage holds at this padded rank.
inline int stage_cols(int stage_bytes, int rp) { return (stage_bytes / (2 * rp)) & ~127; }

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
  const bool small = stage_cols(ShapeSmall::kStageBytes, a.rp) >= 128;
  const int n_warps = small ? ShapeSmall::kWarps : ShapeLarge::kWarps;
  a.stage_bytes = small ? ShapeSmall::kStageBytes : ShapeLarge::kStageBytes;
  a.cols = stage_cols(a.stage_bytes, a.rp);
  if (a.cols < 128) return MILORA_E_SHAPE;
  // a buffer: the stage, then kR rows of x; the smallest padded rank (16) gives the widest rows
  a.buf_stride = (a.stage_bytes + kR * (a.cols * 2 + kRowPad) + 127) & ~127;
  double stages_per_job = 0;
  for (int m = 0; m < MILORA_NMOD; ++m) {
    module_dims(ctx->desc, m, &a.d1[m], &a.d2[m]);
    stages_per_job += ((a.d1[m] + a.cols - 1) / a.cols + (a.d2[m] + a.cols - 1) / a.cols) / (double)MILORA_NMOD;
  }
  const int workers = ctx->sm_count * n_warps;
  int us = ctx->stream_unit_stages;
  if (us < 1) {
    // A unit costs its worker's scheduler lane a round (locate, fetch and decode the job record) and the job a
    // partial sum, so units are several stages long as soon as there are stages enough for every worker: single
    // stages while there is less than one per worker, then two, four, and eight from six stages per worker on
    // (measured on 1 to 32 layers of the 7B shapes at 64 rows and on the 13B shapes at 256).
    const double est = stages_per_job * std::max(1, n_seq_hint) * std::min(n_layers, kMaxStreamLayers);
    const double per_worker = est / workers;
    us = per_worker < 1.0 ? 1 : (per_worker < 2.0 ? 2 : (per_worker < 6.0 ? 4 : 8));
  }
  a.unit_stages = us;
  int kcmax = 1;
  for (int m = 0; m < MILORA_NMOD; ++m)
    kcmax = std::max(kcmax, ((a.d1[m] + a.cols - 1) / a.cols + us - 1) / us);
  a.kcmax = kcmax;
  const size_t frag_bytes = (size_t)(a.rp >> 4) * 32 * sizeof(uint4);
  const size_t part_bytes = (size_t)kcmax * kR * a.rp * sizeof(uint2);
  // scratch of a launch: control words | job states | fragments | partial sums
  auto scratch_bytes = [&](size_t jobs) { return 256 + align256(jobs * 8) + align256(jobs * frag_bytes) + jobs * part_bytes; };
  const size_t cap_bytes = (size_t)512 << 20;
  const size_t smem = (size_t)n_warps * kBufs * a.buf_stride + sizeof(Smem);
  if (!ctx->stream_attr_set) {
    const int top = 227 * 1024;
    MILORA_CUDA(ctx, cudaFuncSetAttribute(decode_stream_kernel<ShapeSmall>, cudaFuncAttributeMaxDynamicSharedMemorySize, top));
    MILORA_CUDA(ctx, cudaFuncSetAttribute(decode_stream_kernel<ShapeLarge>, cudaFuncAttributeMaxDynamicSharedMemorySize, top));
    ctx->stream_attr_set = true;
  }
  if (smem > 227 * 1024) return MILORA_E_SHAPE;

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
    // The buffer is laid out for its capacity (jobs, bytes per job), not for the batch at hand, so a job's counter
    // never serves as anything else; every launch leaves the counters at zero, and they are cleared by the host only
    // when the buffer is new or after a launch that failed or timed out.  Fragments carry the launch's tag.
    if (jobs > ctx->stream_jobs_cap || frag_bytes > ctx->stream_frag_bytes || part_bytes > ctx->stream_part_bytes) {
      const size_t jc = std::max(jobs, ctx->stream_jobs_cap);
      const size_t fb = std::max(frag_bytes, ctx->stream_frag_bytes), pb = std::max(part_bytes, ctx->stream_part_bytes);
      const size_t need = 256 + align256(jc * 8) + align256(jc * fb) + jc * pb;
      MILORA_CUDA(ctx, cudaStreamSynchronize(s));
      if (ctx->d_stream) MILORA_CUDA(ctx, cudaFree(ctx->d_stream));
      ctx->d_stream = nullptr;
      ctx->stream_jobs_cap = 0;
      MILORA_CUDA(ctx, cudaMalloc(&ctx->d_stream, need));
      // fresh memory may hold anything, also words that look like a later launch's tag
      MILORA_CUDA(ctx, cudaMemsetAsync(ctx->d_stream, 0, need, s));
      ctx->stream_jobs_cap = jc;
      ctx->stream_frag_bytes = fb;
      ctx->stream_part_bytes = pb;
      ctx->stream_dirty = true;
    }
    char* base = static_cast<char*>(ctx->d_stream);
    const size_t state_bytes = align256(ctx->stream_jobs_cap * 8);
    a.ctrl = reinterpret_cast<uint32_t*>(base);
    a.job_state = reinterpret_cast<uint32_t*>(base + 256);
    a.vfrag = reinterpret_cast<uint4*>(base + 256 + state_bytes);
    a.partial = reinterpret_cast<uint2*>(base + 256 + state_bytes + align256(ctx->stream_jobs_cap * ctx->stream_frag_bytes));
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
    if (++ctx->stream_epoch == 0) ++ctx->stream_epoch;      // 0 is what a cleared buffer holds
    a.epoch = ctx->stream_epoch;
    ctx->stream_dirty = true;       // stays set if the launch fails
    if (small) {
      MILORA_CUDA(ctx, launch_pdl(decode_stream_kernel<ShapeSmall>, dim3((unsigned)ctx->sm_count), dim3(ShapeSmall::kThreads), smem, s, a));
    } else {
      MILORA_CUDA(ctx, launch_pdl(decode_stream_kernel<ShapeLarge>, dim3((unsigned)ctx->sm_count), dim3(ShapeLarge::kThreads), smem, s, a));
    }
    ctx->stream_dirty = false;
    l0 = l1;
  }
  return MILORA_OK;
}

}  // namespace milora
