// Prefill path of Eq. 1 for bf16 on sm_100a: Y[rows] += s * (X[rows] . A) . B for dense tiles of up to
// 128 consecutive prompt rows that share one adapter.  Both contractions run on the 5th-generation
// tensor cores (tcgen05.mma, accumulators in tensor memory); the op as a whole is bound by streaming
// X once and reading and writing Y once, so the kernels are organised around keeping HBM busy:
//
//   shrink kernel  V_k[rows][r] = X[rows][k-slice] . A[k-slice][r]      one CTA per (tile, k-slice)
//     X tiles arrive by TMA (128-byte swizzle) and the matching A chunks by one bulk copy each
//     (the library keeps A pre-cut into shared-memory operand images) through a 6-stage ring;
//     one thread issues 128 x r x 16 MMAs; the fp32 partial result goes to a small scratch.
//   expand kernel  Y[rows][n-slice] += s * (sum_k V_k) . B[r][n-slice]   one CTA per (tile, n-slice)
//     the summed V (rounded to bf16) is the shared-memory A operand; per 128-column chunk a TMA load
//     brings Y and a bulk copy brings the B image, one MMA chain writes the delta to tensor memory
//     (double buffered), the epilogue warps add it to Y in shared memory and a TMA store writes it
//     back.  Tiles with fewer than 128 rows store their rows with plain 128-bit stores instead, so
//     rows of neighbouring sequences are never touched.
//
// Splitting k and n over CTAs keeps all SMs busy even when a call covers only a few tiles; the partial
// sums are added in k order, so the result does not depend on scheduling.  Every wait is bounded.
#include <cuda.h>

#include "milora_internal.h"
#include "sm100_ptx.cuh"

namespace milora {
namespace {

using namespace ptx;

constexpr int kKSplit = 4;            // k-slices of the shrink
constexpr int kNSplit = 8;            // n-slices of the expand
constexpr int kBK = 64;               // k elements per shrink stage (128 bytes: one swizzle row)
constexpr int kBN = 128;              // y columns per expand chunk
constexpr int kRPadMax = 64;          // largest padded rank this path takes
constexpr int kShrinkStages = 6;
constexpr int kExpandStages = 3;
constexpr int kXStage = kTileRows * kBK * 2;    // 16 KiB
constexpr int kYStage = kTileRows * kBN * 2;    // 32 KiB (two 64-column TMA boxes)
constexpr int kShrinkThreads = 128;
constexpr int kExpandThreads = 192;             // warp 0 copies, warp 1 issues MMAs, warps 2..5 epilogue
constexpr int kIdentBytes = 16 * 16 * 2;        // expand: identity block that carries y into the accumulator

struct PrefillSites {
  int module[kMaxSites], d1[kMaxSites], d2[kMaxSites];
  void* Y[kMaxSites];
  int n;
};

struct ShrinkArgs {
  CUtensorMap xmap[kMaxSites];
  PrefillSites sites;
  int32_t* err;
  const int32_t* ws;
  milora_group_layout_t lay;
  float* vscratch;     // [kKSplit][max_tiles * 128][rpad]: indexed by tile, since with top-k routing a row sits in several tiles
  int T, rpad;
  // shared-input variant only
  int share[kMaxSites];        // sites with equal values read the same X matrix
  int K, n_ent, stages;        // selected modules per sequence, entries of the batch, depth of the copy ring
};

struct ExpandArgs {
  CUtensorMap ymap[kMaxSites];
  PrefillSites sites;
  int32_t* err;
  const int32_t* ws;
  milora_group_layout_t lay;
  const float* vscratch;
  int T, rpad;
};

__device__ __forceinline__ int find_site(const PrefillSites& s, int module) {
  int si = -1;
#pragma unroll
  for (int i = 0; i < kMaxSites; ++i)
    if (i < s.n && s.module[i] == module) si = i;
  return si;
}

// Bounded wait that also gives up as soon as another thread of the CTA has raised `abort`.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort, int32_t* err) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63) == 63 && *abort) return false;
  }
  *abort = 1;
  atomicOr(err, ERR_WAIT_TIMEOUT);
  return false;
}

// After a wait has run out (`abort` is set) copies that were started may still be on their way into this CTA's
// shared memory.  The thread that started them gives every ring stage one more, equally bounded, wait for the last
// phase it asked for, so that whatever is merely late has landed before the CTA frees its tensor memory and leaves.
// `issued` copies went to stages 0, 1, ... in turn; full(s) is the barrier of stage s.
template <class FullOf>
__device__ __forceinline__ void drain_ring(volatile int* abort, int issued, int stages, FullOf full) {
  if (!*abort) return;
  for (int s = 0; s < stages && s < issued; ++s) {
    const int last = ((issued - 1 - s) / stages) * stages + s;      // last copy that went to stage s
    mbar_wait(full(s), (uint32_t)(last / stages) & 1u);
  }
}

__device__ __forceinline__ uint32_t tmem_cols_for(int rp) { return rp <= 32 ? 32u : 64u; }

// ------------------------------------------------------------------------------------------------------
// shrink
// ------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kShrinkThreads) prefill_shrink_kernel(const __grid_constant__ ShrinkArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ks = blockIdx.x % kKSplit;
  // The expand kernel starts its copies of y and B before its own wait; it may do so only once
  // everything ahead of this kernel has completed, so the trigger comes after the wait here.
  pdl_wait();
  pdl_launch_dependents();
  // The tile list is ordered by module and the modules with the longest rows (gate, up, down) come last: CTAs
  // take the list from its end, so that the long tiles start first and the short ones fill the tail.
  const int n_tiles = min(a.ws[a.lay.header + H_NTILES], a.lay.max_tiles);
  const int tile_idx = n_tiles - 1 - (int)(blockIdx.x / kKSplit);
  if (tile_idx < 0) return;
  const TileJob job = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles)[tile_idx];
  const int si = find_site(a.sites, job.module);
  if (si < 0) return;
  const int rp = job.rank_pad;
  const uint32_t base = smem_u32(smem_raw);
  if (!job.At_img || rp < 16 || rp > a.rpad || (rp & 15) || (base & 1023) || job.count < 1 || job.count > kTileRows ||
      job.start < 0 || job.start + job.count > a.T) {
    if (tid == 0) atomicOr(a.err, ERR_BAD_ITEM);
    return;
  }
  const int d1 = a.sites.d1[si];
  const int nchunks = d1 / kBK, cps = (nchunks + kKSplit - 1) / kKSplit;
  const int kc0 = ks * cps, kc1 = min(nchunks, kc0 + cps), nk = max(kc1 - kc0, 0);

  const uint32_t xs = base;
  const uint32_t as = xs + kShrinkStages * kXStage;
  const uint32_t a_stage = (uint32_t)a.rpad * 128u;
  const uint32_t bars = as + kShrinkStages * a_stage;
  auto full = [&](int i) { return bars + 8u * i; };
  auto empty = [&](int i) { return bars + 8u * (kShrinkStages + i); };
  const uint32_t accb = bars + 16u * kShrinkStages;
  const uint32_t slot = accb + 8u;
  volatile uint32_t* slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (slot - base));
  volatile int* abort_ptr = reinterpret_cast<volatile int*>(smem_raw + (slot + 4 - base));
  const uint32_t ncols = tmem_cols_for(rp);

  if (tid == 0) {
    *abort_ptr = 0;
    for (int i = 0; i < kShrinkStages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
    mbar_init(accb, 1);
    fence_barrier_init();
    prefetch_tensormap(&a.xmap[si]);
  }
  __syncthreads();
  if (warp == 0) { tmem_alloc(slot, ncols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *slot_ptr;

  int issued = 0;       // copies started by this thread (the copy thread only)
  if (nk > 0) {
    if (warp == 0 && lane == 0) {
      // ---- copies: X tile by TMA, A image chunk by one bulk copy ----
      const char* img = static_cast<const char*>(job.At_img);
      const uint64_t pol_x = l2_evict_first_policy();      // x is read once; the A images are read again by other tiles
      for (int i = 0; i < nk; ++i) {
        const int s = i % kShrinkStages, ph = (i / kShrinkStages) & 1;
        if (i >= kShrinkStages && !wait_bar(empty(s), ph ^ 1, abort_ptr, a.err)) break;
        mbar_expect_tx(full(s), kXStage + rp * 128);
        tma_load_2d_hint(xs + s * kXStage, &a.xmap[si], (kc0 + i) * kBK, job.start, full(s), pol_x);
        bulk_g2s(as + s * a_stage, img + (size_t)(kc0 + i) * rp * 128, rp * 128, full(s));
        issued = i + 1;
      }
    } else if (warp == 1 && lane == 0) {
      // ---- MMAs: D[128 x rp] += X[128 x 16] * A[16 x rp], four per stage ----
      const uint32_t idesc = idesc_bf16_f32(kTileRows, rp);
      const uint32_t lbo = (uint32_t)(rp / 8) * 128u;        // A image: k-adjacent core matrices
      bool ok = true;
      for (int i = 0; i < nk && ok; ++i) {
        const int s = i % kShrinkStages, ph = (i / kShrinkStages) & 1;
        ok = wait_bar(full(s), ph, abort_ptr, a.err);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kBK / 16; ++kk) {
          const uint64_t da = smem_desc(xs + s * kXStage + kk * 32, 16, 1024, 2);
          const uint64_t db = smem_desc(as + s * a_stage + kk * 2 * lbo, lbo, 128, 0);
          mma_bf16_ss(tmem_base, da, db, idesc, (i | kk) != 0);
        }
        mma_commit(empty(s));
      }
      mma_commit(accb);
    }
  }
  __syncwarp();

  // ---- epilogue: fp32 partial product to the scratch ----
  bool ok = true;
  if (nk > 0) ok = wait_bar(accb, 0, abort_ptr, a.err);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  const int m = warp * 32 + lane;
  float* dst = a.vscratch + (((size_t)ks * a.lay.max_tiles + tile_idx) * kTileRows + m) * a.rpad;
  for (int c0 = 0; c0 < rp; c0 += 16) {
    uint32_t v[16];
    if (nk > 0 && ok) {
      tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + c0, v);
      tmem_wait_ld();
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = 0u;
    }
    if (m < job.count) {
#pragma unroll
      for (int i = 0; i < 16; i += 4)
        *reinterpret_cast<uint4*>(dst + c0 + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    }
  }
  if (warp == 0 && lane == 0) drain_ring(abort_ptr, issued, kShrinkStages, full);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, ncols);
}

// ------------------------------------------------------------------------------------------------------
// shrink, shared input
// ------------------------------------------------------------------------------------------------------
// With top-k routing (Section 3.3 allows k > 1) a sequence selects several modules of a layer, and q, k, v (or gate
// and up) read the same X.  Every selected module has its own tiles over the sequence's rows; tile r of each
// sibling covers the same 128 rows.  Here one CTA takes up to kMaxShare sibling tiles at once: every X stage is
// copied once and multiplied with each sibling's A image into its own tensor-memory columns.  The sibling with
// the lowest module number leads; the CTAs of the others return at once.  The
// partial products land where the plain shrink kernel would have put them, so the expand kernel does not change.
constexpr int kMaxShare = 3;

__device__ __forceinline__ uint32_t tmem_cols_pow2(int cols) {
  uint32_t c = 32;
  while ((int)c < cols) c <<= 1;
  return c;
}

__global__ void __launch_bounds__(kShrinkThreads) prefill_shrink_shared_kernel(const __grid_constant__ ShrinkArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ks = blockIdx.x % kKSplit;
  pdl_wait();
  pdl_launch_dependents();
  const int n_tiles = min(a.ws[a.lay.header + H_NTILES], a.lay.max_tiles);
  const int tile_idx = n_tiles - 1 - (int)(blockIdx.x / kKSplit);
  if (tile_idx < 0) return;
  const TileJob* tiles = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles);
  const TileJob job = tiles[tile_idx];
  const int si = find_site(a.sites, job.module);
  if (si < 0) return;
  const uint32_t base = smem_u32(smem_raw);
  const int stages = a.stages;
  const int ent = job.ent & 0xffff, tiled = (job.ent >> 16) & 0x7f;
  bool bad = (base & 1023) || ent >= a.n_ent || job.module < 0 || job.module >= MILORA_NMOD || !(tiled >> job.module & 1) ||
             job.count < 1 || job.count > kTileRows || job.start < 0 || job.start + job.count > a.T || stages < 2;
  if (bad) {
    if (tid == 0) atomicOr(a.err, ERR_BAD_ITEM);
    return;
  }
  // ---- the siblings: modules with tiles for this sequence whose site reads the same X, by module number; the
  // record of the tile says which modules those are, so a CTA that does not lead leaves without another load ----
  int sib = 0;
#pragma unroll
  for (int m = 0; m < MILORA_NMOD; ++m) {
    const int sj = find_site(a.sites, m);
    if ((tiled >> m & 1) && sj >= 0 && a.share[sj] == a.share[si]) sib |= 1 << m;
  }
  if (__popc(sib & ((1 << job.module) - 1)) % kMaxShare) return;      // an earlier sibling leads this tile
  int mem_mod[kMaxShare], mem_tile[kMaxShare];
  int n_mem = 0;
#pragma unroll
  for (int m = 0; m < MILORA_NMOD; ++m)
    if (m >= job.module && (sib >> m & 1) && n_mem < kMaxShare) mem_mod[n_mem++] = m;
  const int32_t* seq_tile = a.ws + a.lay.seq_tile + 8 * (size_t)(ent / a.K);
#pragma unroll
  for (int m = 0; m < kMaxShare; ++m) mem_tile[m] = m < n_mem ? seq_tile[mem_mod[m]] : -1;
  const int r = tile_idx - mem_tile[0];                 // this tile's position among the tiles of its sequence
  bad = mem_tile[0] < 0 || r < 0;

  const void* img[kMaxShare];
  int rp[kMaxShare], col[kMaxShare];
  TileJob sjob[kMaxShare];
#pragma unroll
  for (int m = 0; m < kMaxShare; ++m) {
    const int t = mem_tile[m] + r;
    bad = bad || (m < n_mem && (mem_tile[m] < 0 || t >= n_tiles));
    mem_tile[m] = t;
    if (m > 0 && m < n_mem && !bad) sjob[m] = tiles[t];
  }
  sjob[0] = job;
  int cols = 0;
#pragma unroll
  for (int m = 0; m < kMaxShare; ++m) {
    img[m] = nullptr; rp[m] = 0; col[m] = cols;
    if (m < n_mem && !bad) {
      img[m] = sjob[m].At_img;
      rp[m] = sjob[m].rank_pad;
      bad = bad || !img[m] || rp[m] < 16 || rp[m] > a.rpad || (rp[m] & 15) || sjob[m].start != job.start ||
            sjob[m].count != job.count || sjob[m].module != mem_mod[m];
      cols += rp[m];
    }
  }
  if (bad) {
    if (tid == 0) atomicOr(a.err, ERR_BAD_ITEM);
    return;
  }
  const int d1 = a.sites.d1[si];
  const int nchunks = d1 / kBK, cps = (nchunks + kKSplit - 1) / kKSplit;
  const int kc0 = ks * cps, kc1 = min(nchunks, kc0 + cps), nk = max(kc1 - kc0, 0);

  const uint32_t xs = base;
  const uint32_t as = xs + stages * kXStage;
  const uint32_t a_one = (uint32_t)a.rpad * 128u;           // one sibling's A chunk
  const uint32_t a_stage = kMaxShare * a_one;
  const uint32_t bars = as + stages * a_stage;
  auto full = [&](int i) { return bars + 8u * i; };
  auto empty = [&](int i) { return bars + 8u * (stages + i); };
  const uint32_t accb = bars + 16u * stages;
  const uint32_t slot = accb + 8u;
  volatile uint32_t* slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (slot - base));
  volatile int* abort_ptr = reinterpret_cast<volatile int*>(smem_raw + (slot + 4 - base));
  const uint32_t ncols = tmem_cols_pow2(cols);

  if (tid == 0) {
    *abort_ptr = 0;
    for (int i = 0; i < stages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), n_mem); }
    mbar_init(accb, n_mem);
    fence_barrier_init();
    prefetch_tensormap(&a.xmap[si]);
  }
  __syncthreads();
  if (warp == 0) { tmem_alloc(slot, ncols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *slot_ptr;

  // One thread starts a copy or an MMA every fifty to a hundred cycles, and a stage arrives from memory about every
  // 1400: the copies of a stage (X tile, one A chunk per sibling) stay with one thread, and every sibling's four
  // MMAs get a thread of their own (warps 1, 2, 3), each of which commits to the stage's `empty` barrier.
  int issued = 0;
  if (nk > 0) {
    if (warp == 0) {
      if (lane == 0) {
        // ---- copies: the X tile once (read once: evict first), one A image chunk per sibling ----
        const uint64_t pol_x = l2_evict_first_policy();
        for (int i = 0; i < nk; ++i) {
          const int s = i % stages, ph = (i / stages) & 1;
          if (i >= stages && !wait_bar(empty(s), ph ^ 1, abort_ptr, a.err)) break;
          mbar_expect_tx(full(s), kXStage + cols * 128);
          tma_load_2d_hint(xs + s * kXStage, &a.xmap[si], (kc0 + i) * kBK, job.start, full(s), pol_x);
#pragma unroll
          for (int m = 0; m < kMaxShare; ++m)
            if (m < n_mem)
              bulk_g2s(as + s * a_stage + m * a_one, static_cast<const char*>(img[m]) + (size_t)(kc0 + i) * rp[m] * 128,
                       rp[m] * 128, full(s));
          issued = i + 1;
        }
      }
    } else if (lane == 0 && warp - 1 < n_mem) {
      // ---- MMAs of sibling warp - 1: D_m[128 x rp_m] += X[128 x 16] * A_m[16 x rp_m], four per stage ----
      int rp_m = 0, col_m = 0;
#pragma unroll
      for (int m = 0; m < kMaxShare; ++m)
        if (m == warp - 1) { rp_m = rp[m]; col_m = col[m]; }
      const uint32_t idesc = idesc_bf16_f32(kTileRows, rp_m);
      const uint32_t lbo = (uint32_t)(rp_m / 8) * 128u;        // A image: k-adjacent core matrices
      const uint32_t a_m = as + (uint32_t)(warp - 1) * a_one;
      bool ok = true;
      for (int i = 0; i < nk && ok; ++i) {
        const int s = i % stages, ph = (i / stages) & 1;
        ok = wait_bar(full(s), ph, abort_ptr, a.err);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kBK / 16; ++kk) {
          const uint64_t da = smem_desc(xs + s * kXStage + kk * 32, 16, 1024, 2);
          const uint64_t db = smem_desc(a_m + s * a_stage + kk * 2 * lbo, lbo, 128, 0);
          mma_bf16_ss(tmem_base + col_m, da, db, idesc, (i | kk) != 0);
        }
        mma_commit(empty(s));
      }
      mma_commit(accb);
    }
  }
  __syncwarp();

  // ---- epilogue: every sibling's fp32 partial product to its own tile of the scratch ----
  bool ok = true;
  if (nk > 0) ok = wait_bar(accb, 0, abort_ptr, a.err);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  const int row = warp * 32 + lane;
#pragma unroll
  for (int m = 0; m < kMaxShare; ++m) {
    if (m >= n_mem) continue;
    float* dst = a.vscratch + (((size_t)ks * a.lay.max_tiles + mem_tile[m]) * kTileRows + row) * a.rpad;
    for (int c0 = 0; c0 < rp[m]; c0 += 16) {
      uint32_t v[16];
      if (nk > 0 && ok) {
        tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + col[m] + c0, v);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = 0u;
      }
      if (row < job.count) {
#pragma unroll
        for (int i = 0; i < 16; i += 4)
          *reinterpret_cast<uint4*>(dst + c0 + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
      }
    }
  }
  if (warp == 0 && lane == 0) drain_ring(abort_ptr, issued, stages, full);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, ncols);
}

// ------------------------------------------------------------------------------------------------------
// expand
// ------------------------------------------------------------------------------------------------------
// Eight fp32 accumulator values (y + delta) rounded to bf16.
__device__ __forceinline__ uint4 pack8(const uint32_t* d) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(d[2 * i]), __uint_as_float(d[2 * i + 1]));
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(kExpandThreads) prefill_expand_kernel(const __grid_constant__ ExpandArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ns = blockIdx.x % kNSplit;
  // Launched behind the shrink kernel, whose CTAs trigger only after their own wait: the job list, y and
  // the B images are final when this CTA starts.  Only the partial products of the shrink need pdl_wait().
  pdl_launch_dependents();
  const int n_tiles = min(a.ws[a.lay.header + H_NTILES], a.lay.max_tiles);
  const int tile_idx = n_tiles - 1 - (int)(blockIdx.x / kNSplit);       // longest tiles first, as in the shrink kernel
  if (tile_idx < 0) { pdl_wait(); return; }
  const TileJob job = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles)[tile_idx];
  const int si = find_site(a.sites, job.module);
  if (si < 0) { pdl_wait(); return; }
  const int rp = job.rank_pad;
  const uint32_t base = smem_u32(smem_raw);
  if (!job.B_img || rp < 16 || rp > a.rpad || (rp & 15) || (base & 1023) || job.count < 1 || job.count > kTileRows ||
      job.start < 0 || job.start + job.count > a.T) {
    if (tid == 0) atomicOr(a.err, ERR_BAD_ITEM);
    pdl_wait();
    return;
  }
  const int d2 = a.sites.d2[si];
  const int nchunks = d2 / kBN, cps = (nchunks + kNSplit - 1) / kNSplit;
  const int nc0 = ns * cps, nc1 = min(nchunks, nc0 + cps), nn = nc1 - nc0;
  if (nn <= 0) { pdl_wait(); return; }

  const uint32_t ys = base;
  const uint32_t bs = ys + kExpandStages * kYStage;
  const uint32_t b_stage = (uint32_t)a.rpad * 256u;
  const uint32_t vs = bs + kExpandStages * b_stage;
  const uint32_t ident = vs + (uint32_t)kTileRows * a.rpad * 2u;     // 16 x 16 identity, 512 bytes
  const uint32_t bars = ident + kIdentBytes;
  auto full = [&](int i) { return bars + 8u * i; };
  auto empty = [&](int i) { return bars + 8u * (kExpandStages + i); };
  auto tfull = [&](int i) { return bars + 8u * (2 * kExpandStages + i); };
  auto tempty = [&](int i) { return bars + 8u * (2 * kExpandStages + 2 + i); };
  const uint32_t slot = bars + 8u * (2 * kExpandStages + 4);
  volatile uint32_t* slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (slot - base));
  volatile int* abort_ptr = reinterpret_cast<volatile int*>(smem_raw + (slot + 4 - base));
  constexpr uint32_t kCols = 2 * kBN;

  if (tid == 0) {
    *abort_ptr = 0;
    for (int i = 0; i < kExpandStages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull(i), 1); mbar_init(tempty(i), 128); }
    fence_barrier_init();
    prefetch_tensormap(&a.ymap[si]);
  }
  __syncthreads();
  const int row0 = job.start;
  int issued = 0;                       // copies started by this thread (the copy thread only)
  const uint64_t pol_y = l2_evict_first_policy();       // y is read once; the B images are read again by other tiles
  auto issue_stage = [&](int i) {       // y tile (two 64-column boxes) and B image chunk of n chunk i
    const int s = i % kExpandStages;
    mbar_expect_tx(full(s), kYStage + rp * 256);
    tma_load_2d_hint(ys + s * kYStage, &a.ymap[si], (nc0 + i) * kBN, row0, full(s), pol_y);
    tma_load_2d_hint(ys + s * kYStage + kYStage / 2, &a.ymap[si], (nc0 + i) * kBN + 64, row0, full(s), pol_y);
    bulk_g2s(bs + s * b_stage, static_cast<const char*>(job.B_img) + (size_t)(nc0 + i) * rp * 256, rp * 256, full(s));
  };
  if (warp == 0) {
    tmem_alloc(slot, kCols);
    tmem_relinquish();
    // first pass over the ring: these copies do not depend on the shrink kernel
    if (lane == 0)
      for (int i = 0; i < nn && i < kExpandStages; ++i) issue_stage(i);
      issued = min(nn, kExpandStages);
  }

  // epilogue threads also build the A operand: V = s * sum_k V_k, bf16, 8 x 16-byte core-matrix rows
  const int q = warp & 3;               // tensor-memory lane quarter this warp may read
  const int m = q * 32 + lane;          // row of the tile this thread owns
  if (warp >= 2) {
    pdl_wait();                         // the partial products written by the shrink kernel
    unsigned char* vrow = smem_raw + (vs - base) + (size_t)(m >> 3) * 128 + (size_t)(m & 7) * 16;
    for (int c0 = 0; c0 < rp; c0 += 8) {
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.f;
      if (m < job.count) {
#pragma unroll
        for (int k = 0; k < kKSplit; ++k) {
          const float4* src =
              reinterpret_cast<const float4*>(
                  a.vscratch + (((size_t)k * a.lay.max_tiles + tile_idx) * kTileRows + m) * a.rpad + c0);
          const float4 u0 = __ldcg(src), u1 = __ldcg(src + 1);
          acc[0] += u0.x; acc[1] += u0.y; acc[2] += u0.z; acc[3] += u0.w;
          acc[4] += u1.x; acc[5] += u1.y; acc[6] += u1.z; acc[7] += u1.w;
        }
      }
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i] * job.scale, acc[2 * i + 1] * job.scale);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(vrow + (size_t)(c0 >> 3) * (kTileRows / 8) * 128) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    // I_16 as a K-major operand without swizzle: core matrix (n / 8, k / 8) at ((k / 8) * 2 + n / 8) * 128 bytes
    for (int idx = tid - 64; idx < 256; idx += 128) {
      const int n = idx >> 4, k = idx & 15;
      const uint32_t off = (uint32_t)(((k >> 3) * 2 + (n >> 3)) * 128 + (n & 7) * 16 + (k & 7) * 2);
      *reinterpret_cast<unsigned short*>(smem_raw + (ident - base) + off) = (n == k) ? 0x3F80 : 0;   // bf16 1.0
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *slot_ptr;
  const bool full_tile = job.count == kTileRows;

  if (warp == 0) {
    if (lane == 0) {
      for (int i = kExpandStages; i < nn; ++i) {
        const int s = i % kExpandStages, ph = (i / kExpandStages) & 1;
        if (!wait_bar(empty(s), ph ^ 1, abort_ptr, a.err)) break;
        issue_stage(i);
        issued = i + 1;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kTileRows, kBN);
      const uint32_t idesc_i = idesc_bf16_f32(kTileRows, 16);
      const uint64_t di = smem_desc(ident, 256, 128, 0);
      constexpr uint32_t kLbo = (kTileRows / 8) * 128u;      // both operands: 16 core matrices per k group
      for (int i = 0; i < nn; ++i) {
        const int s = i % kExpandStages, ph = (i / kExpandStages) & 1, b = i & 1, bph = (i >> 1) & 1;
        if (!wait_bar(full(s), ph, abort_ptr, a.err)) break;
        if (i >= 2 && !wait_bar(tempty(b), bph ^ 1, abort_ptr, a.err)) break;
        tc_fence_after();
        for (int kk = 0; kk < rp / 16; ++kk) {
          const uint64_t da = smem_desc(vs + kk * 2 * kLbo, kLbo, 128, 0);
          const uint64_t db = smem_desc(bs + s * b_stage + kk * 2 * kLbo, kLbo, 128, 0);
          mma_bf16_ss(tmem_base + b * kBN, da, db, idesc, kk != 0);
        }
        // y itself joins the accumulator: D[:, 16g .. 16g+16) += Y[:, 16g .. 16g+16) . I_16 (exact in fp32),
        // so the epilogue only converts and stores.  The y tile is the 128-byte-swizzled K-major A operand.
#pragma unroll
        for (int g = 0; g < kBN / 16; ++g) {
          const uint64_t da = smem_desc(ys + s * kYStage + (g >> 2) * (kYStage / 2) + (g & 3) * 32, 16, 1024, 2);
          mma_bf16_ss(tmem_base + b * kBN + g * 16, da, di, idesc_i, 1);
        }
        mma_commit(tfull(b));
      }
    }
  } else {
    const int e = tid - 64;
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(a.sites.Y[si]);
    bool ok = true;
    for (int i = 0; i < nn && ok; ++i) {
      const int s = i % kExpandStages, ph = (i / kExpandStages) & 1, b = i & 1, bph = (i >> 1) & 1;
      ok = wait_bar(tfull(b), bph, abort_ptr, a.err) && wait_bar(full(s), ph, abort_ptr, a.err);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      unsigned char* ytile = smem_raw + (ys - base) + (size_t)s * kYStage;
      // 64 columns (one 128-byte swizzle box of y) per round: two tensor-memory loads in flight, one wait
#pragma unroll 1
      for (int box = 0; box < kBN / 64; ++box) {
        uint32_t d0[32], d1v[32];
        const uint32_t taddr = tmem_base + b * kBN + ((uint32_t)(q * 32) << 16) + box * 64;
        tmem_ld32(taddr, d0);
        tmem_ld32(taddr + 32, d1v);
        tmem_wait_ld();
        if (m < job.count) {
          unsigned char* yrow = ytile + (size_t)box * (kYStage / 2) + (size_t)m * 128;
#pragma unroll
          for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(yrow + ((c ^ (m & 7)) << 4)) = pack8(d0 + 8 * c);
#pragma unroll
          for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(yrow + (((c + 4) ^ (m & 7)) << 4)) = pack8(d1v + 8 * c);
        }
      }
      tc_fence_before();
      mbar_arrive(tempty(b));
      fence_proxy_async_smem();
      named_barrier(1, 128);
      if (full_tile) {
        if (e == 0) {
          tma_store_2d(&a.ymap[si], (nc0 + i) * kBN, row0, ys + s * kYStage);
          tma_store_2d(&a.ymap[si], (nc0 + i) * kBN + 64, row0, ys + s * kYStage + kYStage / 2);
          bulk_commit_group();
          bulk_wait_group_read0();
          mbar_arrive(empty(s));
        }
      } else {
        // a tile with fewer than 128 rows: write only its own rows
        for (int idx = e; idx < job.count * 16; idx += 128) {
          const int rr = idx >> 4, cg = idx & 15, box = cg >> 3, c = cg & 7;
          const uint4 y = *reinterpret_cast<const uint4*>(ytile + (size_t)box * (kYStage / 2) + (size_t)rr * 128 +
                                                          ((c ^ (rr & 7)) << 4));
          *reinterpret_cast<uint4*>(Y + (size_t)(row0 + rr) * d2 + (size_t)(nc0 + i) * kBN + cg * 8) = y;
        }
        named_barrier(1, 128);
        if (e == 0) mbar_arrive(empty(s));
      }
    }
    if (e == 0) bulk_wait_group0();
  }
  __syncwarp();
  pdl_wait();                           // returns at once here; keeps "every thread waited before it exits" true
  if (warp == 0 && lane == 0) drain_ring(abort_ptr, issued, kExpandStages, full);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kCols);
}

// ------------------------------------------------------------------------------------------------------
// fused projection: Y = X . W + b + s (X A) B on the routed rows   (Eq. 1 in one pass over Y)
// ------------------------------------------------------------------------------------------------------
// A persistent tensor-core GEMM over 128 x 256 output tiles (both operands K-major bf16, 64-element k steps
// through a 4-stage TMA ring, two 256-column accumulators in tensor memory so that the epilogue of one tile
// overlaps the main loop of the next).  The LoRA term rides on the same accumulator: after the k loop of a
// tile, every dense LoRA tile that overlaps the tile's 128 rows contributes one more short MMA chain
// V_piece (128 x rank, rows outside the overlap zero) . B (rank x 256).  V comes from the shrink kernel; a
// small kernel packs it, per (LoRA tile, row block) piece, into the shared-memory operand image and lists the
// pieces of every row block.  Y is written once and never read.
constexpr int kLinBM = 128, kLinBN = 256, kLinBK = 64;
constexpr int kLinStages = 4;
constexpr int kLinAStage = kLinBM * kLinBK * 2;   // 16 KiB
constexpr int kLinBStage = kLinBN * kLinBK * 2;   // 32 KiB
constexpr int kLinThreads = 192;                  // warp 0 copies, warp 1 issues MMAs, warps 2..5 epilogue
constexpr int kLinRPadMax = 32;
constexpr int kMaxPieces = 12;                    // LoRA tile pieces that can overlap one block of 128 rows
constexpr int kLinGroupM = 16;                    // row blocks per raster group (their X panels stay in L2)

struct PackArgs {
  int32_t* err;
  const int32_t* ws;
  milora_group_layout_t lay;
  const float* vscratch;
  unsigned char* vimg;       // [max_tiles][2][128 * rpad * 2 bytes]
  int32_t* piece_cnt;        // [n_mblk], zero on entry
  int32_t* piece_job;        // [n_mblk][kMaxPieces]: tile index * 2 + half
  int module, T, rpad, n_mblk;
};

// One CTA per dense LoRA tile of the module: V = s * sum_k V_k rounded to bf16, written as the K-major operand
// image (core matrix (row / 8, k / 8) at ((k / 8) * 16 + row / 8) * 128 bytes) of each of the (at most two)
// 128-row blocks the tile overlaps, and the piece is appended to the block's list.
__global__ void __launch_bounds__(kTileRows) linear_vpack_kernel(PackArgs a) {
  const int tile_idx = blockIdx.x, m = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  const int n_tiles = a.ws[a.lay.header + H_NTILES];
  if (tile_idx >= n_tiles || tile_idx >= a.lay.max_tiles) return;
  const TileJob job = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles)[tile_idx];
  if (job.module != a.module) return;
  const int rp = job.rank_pad;
  if (rp < 16 || rp > a.rpad || (rp & 15) || job.count < 1 || job.count > kTileRows || job.start < 0 ||
      job.start + job.count > a.T) {
    if (m == 0) atomicOr(a.err, ERR_BAD_ITEM);
    return;
  }
  const size_t img_bytes = (size_t)kTileRows * a.rpad * 2;
  unsigned char* img0 = a.vimg + (size_t)tile_idx * 2 * img_bytes;
  for (int i = m; i < (int)(2 * img_bytes / 16); i += kTileRows) reinterpret_cast<uint4*>(img0)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  const int b0 = job.start / kTileRows;
  if (m < job.count) {
    const int row = job.start + m, h = row / kTileRows - b0, rb = row % kTileRows;
    unsigned char* vrow = img0 + (size_t)h * img_bytes + (size_t)(rb >> 3) * 128 + (size_t)(rb & 7) * 16;
    for (int c0 = 0; c0 < rp; c0 += 8) {
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
      for (int k = 0; k < kKSplit; ++k) {
        const float4* src = reinterpret_cast<const float4*>(
            a.vscratch + (((size_t)k * a.lay.max_tiles + tile_idx) * kTileRows + m) * a.rpad + c0);
        const float4 u0 = __ldcg(src), u1 = __ldcg(src + 1);
        acc[0] += u0.x; acc[1] += u0.y; acc[2] += u0.z; acc[3] += u0.w;
        acc[4] += u1.x; acc[5] += u1.y; acc[6] += u1.z; acc[7] += u1.w;
      }
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 hh = __floats2bfloat162_rn(acc[2 * i] * job.scale, acc[2 * i + 1] * job.scale);
        w[i] = *reinterpret_cast<uint32_t*>(&hh);
      }
      *reinterpret_cast<uint4*>(vrow + (size_t)(c0 >> 3) * (kTileRows / 8) * 128) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
  if (m == 0) {
    for (int h = 0; h < 2; ++h) {
      const int b = b0 + h;
      const int lo = max(job.start, b * kTileRows), hi = min(job.start + job.count, (b + 1) * kTileRows);
      if (lo >= hi || b >= a.n_mblk) continue;
      const int slot = atomicAdd(&a.piece_cnt[b], 1);
      if (slot < kMaxPieces) a.piece_job[b * kMaxPieces + slot] = tile_idx * 2 + h;
      else atomicOr(a.err, ERR_BAD_ITEM);
    }
  }
}

struct LinearArgs {
  CUtensorMap xmap, wmap;
  int32_t* err;
  const int32_t* ws;
  milora_group_layout_t lay;
  const unsigned char* vimg;
  const int32_t* piece_cnt;
  const int32_t* piece_job;
  const __nv_bfloat16* bias;   // d2 values or nullptr
  __nv_bfloat16* Y;
  int T, d1, d2, rpad, n_mblk, n_nblk;
};

__global__ void __launch_bounds__(kLinThreads, 1) linear_lora_kernel(const __grid_constant__ LinearArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t as = base;
  const uint32_t bs = as + kLinStages * kLinAStage;
  const uint32_t vs = bs + kLinStages * kLinBStage;                 // V piece image, 128 x rpad bf16
  const uint32_t lbs = vs + (uint32_t)kTileRows * a.rpad * 2u;      // B image, two 128-column chunks
  const uint32_t bars = lbs + (uint32_t)a.rpad * 512u;
  auto full = [&](int i) { return bars + 8u * i; };
  auto empty = [&](int i) { return bars + 8u * (kLinStages + i); };
  auto tfull = [&](int i) { return bars + 8u * (2 * kLinStages + i); };
  auto tempty = [&](int i) { return bars + 8u * (2 * kLinStages + 2 + i); };
  const uint32_t lfull = bars + 8u * (2 * kLinStages + 4), lempty = lfull + 8u;
  const uint32_t slot = lempty + 8u;
  volatile uint32_t* slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (slot - base));
  volatile int* abort_ptr = reinterpret_cast<volatile int*>(smem_raw + (slot + 4 - base));
  constexpr uint32_t kCols = 2 * kLinBN;

  pdl_launch_dependents();
  if (tid == 0) {
    *abort_ptr = 0;
    for (int i = 0; i < kLinStages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull(i), 1); mbar_init(tempty(i), 128); }
    mbar_init(lfull, 1);
    mbar_init(lempty, 1);
    fence_barrier_init();
    prefetch_tensormap(&a.xmap);
    prefetch_tensormap(&a.wmap);
  }
  __syncthreads();
  if (warp == 0) { tmem_alloc(slot, kCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *slot_ptr;
  pdl_wait();

  const int total = a.n_mblk * a.n_nblk, nk = a.d1 / kLinBK;
  const int per_group = kLinGroupM * a.n_nblk;
  auto tile_coords = [&](int t, int& mb, int& nb) {
    const int g = t / per_group, r = t % per_group;
    const int m0 = g * kLinGroupM;
    const int gm = min(kLinGroupM, a.n_mblk - m0);
    nb = r / gm;
    mb = m0 + r % gm;
  };
  const TileJob* tiles = reinterpret_cast<const TileJob*>(a.ws + a.lay.tiles);
  const bool bad = (base & 1023) != 0 || a.rpad > kLinRPadMax;
  int ring_issued = 0, piece_issued = 0;        // copies started by this thread (the copy thread only)
  if (bad && tid == 0) atomicOr(a.err, ERR_BAD_ITEM);

  if (!bad && warp == 0) {
    if (lane == 0) {
      // ---- copies: X and W tiles by TMA through the ring; V piece image and B image by bulk copies ----
      int it = 0, lit = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        int mb, nb;
        tile_coords(t, mb, nb);
        for (int k = 0; k < nk && ok; ++k, ++it) {
          const int s = it % kLinStages, ph = (it / kLinStages) & 1;
          if (it >= kLinStages) ok = wait_bar(empty(s), ph ^ 1, abort_ptr, a.err);
          if (!ok) break;
          mbar_expect_tx(full(s), kLinAStage + kLinBStage);
          tma_load_2d(as + s * kLinAStage, &a.xmap, k * kLinBK, mb * kLinBM, full(s));
          tma_load_2d(bs + s * kLinBStage, &a.wmap, k * kLinBK, nb * kLinBN, full(s));
          ring_issued = it + 1;
        }
        const int np = min(a.piece_cnt[mb], kMaxPieces);
        for (int p = 0; p < np && ok; ++p, ++lit) {
          if (lit >= 1) ok = wait_bar(lempty, (lit - 1) & 1, abort_ptr, a.err);
          if (!ok) break;
          const int pj = a.piece_job[mb * kMaxPieces + p];
          const TileJob job = tiles[pj >> 1];
          const uint32_t rp = (uint32_t)job.rank_pad;
          mbar_expect_tx(lfull, rp * 256u + rp * 512u);
          bulk_g2s(vs, a.vimg + (size_t)pj * ((size_t)kTileRows * a.rpad * 2), rp * 256u, lfull);
          bulk_g2s(lbs, static_cast<const char*>(job.B_img) + (size_t)(2 * nb) * rp * 256u, rp * 512u, lfull);
          piece_issued = lit + 1;
        }
      }
    }
  } else if (!bad && warp == 1) {
    if (lane == 0) {
      // ---- MMAs ----
      const uint32_t idesc = idesc_bf16_f32(kLinBM, kLinBN), idesc_l = idesc_bf16_f32(kLinBM, 128);
      constexpr uint32_t kLbo = (kTileRows / 8) * 128u;
      int it = 0, lit = 0, ti = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++ti) {
        int mb, nb;
        tile_coords(t, mb, nb);
        const int b = ti & 1, bph = (ti >> 1) & 1;
        if (ti >= 2) ok = wait_bar(tempty(b), bph ^ 1, abort_ptr, a.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tmem_base + (uint32_t)b * kLinBN;
        for (int k = 0; k < nk && ok; ++k, ++it) {
          const int s = it % kLinStages, ph = (it / kLinStages) & 1;
          ok = wait_bar(full(s), ph, abort_ptr, a.err);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < kLinBK / 16; ++kk) {
            const uint64_t da = smem_desc(as + s * kLinAStage + kk * 32, 16, 1024, 2);
            const uint64_t db = smem_desc(bs + s * kLinBStage + kk * 32, 16, 1024, 2);
            mma_bf16_ss(dcol, da, db, idesc, (k | kk) != 0);
          }
          mma_commit(empty(s));
        }
        if (!ok) break;
        const int np = min(a.piece_cnt[mb], kMaxPieces);
        for (int p = 0; p < np && ok; ++p, ++lit) {
          const int pj = a.piece_job[mb * kMaxPieces + p];
          const int rp = tiles[pj >> 1].rank_pad;
          ok = wait_bar(lfull, lit & 1, abort_ptr, a.err);
          if (!ok) break;
          tc_fence_after();
          for (int c = 0; c < 2; ++c) {
            for (int kk = 0; kk < rp / 16; ++kk) {
              const uint64_t da = smem_desc(vs + kk * 2 * kLbo, kLbo, 128, 0);
              const uint64_t db = smem_desc(lbs + c * rp * 256 + kk * 2 * kLbo, kLbo, 128, 0);
              mma_bf16_ss(dcol + c * 128, da, db, idesc_l, 1);
            }
          }
          mma_commit(lempty);
        }
        if (!ok) break;
        mma_commit(tfull(b));
      }
    }
  } else if (!bad) {
    // ---- epilogue: accumulator (+ bias) -> bf16 -> y, 64 bytes per thread and 32-column group ----
    const int q = warp & 3;
    const int rt = q * 32 + lane;
    int ti = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++ti) {
      int mb, nb;
      tile_coords(t, mb, nb);
      const int b = ti & 1, bph = (ti >> 1) & 1;
      ok = wait_bar(tfull(b), bph, abort_ptr, a.err);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = mb * kLinBM + rt;
      __nv_bfloat16* yrow = a.Y + (size_t)row * a.d2 + (size_t)nb * kLinBN;
      const uint32_t taddr = tmem_base + (uint32_t)b * kLinBN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < kLinBN; c0 += 64) {
        uint32_t d0[32], d1v[32];
        tmem_ld32(taddr + c0, d0);
        tmem_ld32(taddr + c0 + 32, d1v);
        tmem_wait_ld();
        if (a.bias) {
          const __nv_bfloat16* bp = a.bias + (size_t)nb * kLinBN + c0;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            d0[i] = __float_as_uint(__uint_as_float(d0[i]) + __bfloat162float(bp[i]));
            d1v[i] = __float_as_uint(__uint_as_float(d1v[i]) + __bfloat162float(bp[32 + i]));
          }
        }
        if (row < a.T) {
#pragma unroll
          for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(yrow + c0 + 8 * i) = pack8(d0 + 8 * i);
#pragma unroll
          for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(yrow + c0 + 32 + 8 * i) = pack8(d1v + 8 * i);
        }
      }
      tc_fence_before();
      mbar_arrive(tempty(b));
    }
  }
  __syncwarp();
  if (warp == 0 && lane == 0) {
    drain_ring(abort_ptr, ring_issued, kLinStages, full);
    drain_ring(abort_ptr, piece_issued, 1, [&](int) { return lfull; });
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kCols);
}

// ------------------------------------------------------------------------------------------------------
// registration-time operand images
// ------------------------------------------------------------------------------------------------------
// A image: for every 64-wide k chunk a block of rp x 64 bf16 as 8 x 16-byte core-matrix rows;
// core matrix (j / 8, k / 8) sits at ((k / 8) * (rp / 8) + j / 8) * 128 bytes.  One thread per 16 bytes.
__global__ void pack_a_image_kernel(const __nv_bfloat16* __restrict__ At, uint4* __restrict__ img, int d1, int r, int rp) {
  const size_t n_pieces = (size_t)(d1 / 8) * rp;
  for (size_t p = blockIdx.x * (size_t)blockDim.x + threadIdx.x; p < n_pieces; p += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(p % rp);
    const int k8 = (int)(p / rp);                 // which group of 8 k values
    const int kc = k8 / 8, ki = k8 % 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (j < r) v = *reinterpret_cast<const uint4*>(At + (size_t)j * d1 + (size_t)k8 * 8);
    const size_t off16 = (size_t)kc * (rp * 8) + ((size_t)ki * (rp / 8) + j / 8) * 8 + (j % 8);
    img[off16] = v;
  }
}

// B image: for every 128-wide n chunk a block of 128 x rp bf16 (n rows, k contiguous);
// core matrix (n / 8, k / 8) sits at ((k / 8) * 16 + n / 8) * 128 bytes.  One thread per 16 bytes.
__global__ void pack_b_image_kernel(const __nv_bfloat16* __restrict__ B, uint4* __restrict__ img, int d2, int r, int rp) {
  const size_t n_pieces = (size_t)d2 * (rp / 8);
  for (size_t p = blockIdx.x * (size_t)blockDim.x + threadIdx.x; p < n_pieces; p += (size_t)gridDim.x * blockDim.x) {
    const int n = (int)(p % d2);
    const int ki = (int)(p / d2);
    const int nc = n / kBN, nl = n % kBN;
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int k0 = ki * 8 + 2 * i;
      const unsigned short lo = k0 < r ? __bfloat16_as_ushort(B[(size_t)k0 * d2 + n]) : 0;
      const unsigned short hi = k0 + 1 < r ? __bfloat16_as_ushort(B[(size_t)(k0 + 1) * d2 + n]) : 0;
      w[i] = (uint32_t)lo | ((uint32_t)hi << 16);
    }
    const size_t off16 = (size_t)nc * (rp * 16) + ((size_t)ki * 16 + nl / 8) * 8 + (nl % 8);
    img[off16] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows][cols] bf16 row-major, tiles of box_rows rows x 64 columns, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows = kTileRows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool prefill_images_supported(const milora_ctx* ctx, int d1, int d2, int rank) {
  return ctx->desc.dtype == MILORA_BF16 && d1 % kBK == 0 && d2 % kBN == 0 && rank >= 1 && rank <= kRPadMax;
}

size_t prefill_image_bytes(int d, int rank) { return (size_t)d * ((rank + 15) & ~15) * 2; }

milora_status launch_pack_images(milora_ctx* ctx, const void* At, const void* B, void* At_img, void* B_img, int d1, int d2,
                                 int rank, cudaStream_t s) {
  const int rp = (rank + 15) & ~15;
  const size_t pa = (size_t)(d1 / 8) * rp, pb = (size_t)d2 * (rp / 8);
  pack_a_image_kernel<<<(unsigned)std::min<size_t>((pa + 255) / 256, 4096), 256, 0, s>>>(
      static_cast<const __nv_bfloat16*>(At), static_cast<uint4*>(At_img), d1, rank, rp);
  MILORA_CUDA(ctx, cudaGetLastError());
  pack_b_image_kernel<<<(unsigned)std::min<size_t>((pb + 255) / 256, 4096), 256, 0, s>>>(
      static_cast<const __nv_bfloat16*>(B), static_cast<uint4*>(B_img), d2, rank, rp);
  MILORA_CUDA(ctx, cudaGetLastError());
  return MILORA_OK;
}

// shrink_only: stop after the shrink kernel (the fused projection consumes its partial products itself).
static milora_status launch_prefill(milora_ctx* ctx, const ApplySites& sites, const milora_groups* g, bool shrink_only,
                                    cudaStream_t s) {
  if (ctx->desc.dtype != MILORA_BF16) return MILORA_E_SHAPE;
  const int T = g->T;
  const int rpad = (ctx->desc.max_rank + 15) & ~15;
  if (rpad > kRPadMax || T < kTileRows) return MILORA_E_SHAPE;
  for (int i = 0; i < sites.n; ++i) {
    const ApplySite& st = sites.site[i];
    if (st.d1 % kBK || st.d2 % kBN) return MILORA_E_SHAPE;
    if ((reinterpret_cast<uintptr_t>(st.X) & 15) || (!shrink_only && (reinterpret_cast<uintptr_t>(st.Y) & 15)))
      return MILORA_E_SHAPE;
  }
  const size_t shrink_smem = (size_t)kShrinkStages * (kXStage + rpad * 128) + 128;
  const size_t expand_smem =
      (size_t)kExpandStages * (kYStage + rpad * 256) + (size_t)kTileRows * rpad * 2 + kIdentBytes + 128;
  if (shrink_smem > 220 * 1024 || expand_smem > 220 * 1024) return MILORA_E_SHAPE;

  const milora_group_layout_t lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  const size_t need = (size_t)kKSplit * lay.max_tiles * kTileRows * rpad;
  if (need > ctx->vscratch_floats) {
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    if (ctx->d_vscratch) MILORA_CUDA(ctx, cudaFree(ctx->d_vscratch));
    ctx->d_vscratch = nullptr;
    ctx->vscratch_floats = 0;
    MILORA_CUDA(ctx, cudaMalloc(&ctx->d_vscratch, need * sizeof(float)));
    ctx->vscratch_floats = need;
  }

  ShrinkArgs sa;
  ExpandArgs ea;
  PrefillSites ps;
  ps.n = sites.n;
  for (int i = 0; i < kMaxSites; ++i) { ps.module[i] = -1; ps.d1[i] = ps.d2[i] = 0; ps.Y[i] = nullptr; }
  for (int i = 0; i < sites.n; ++i) {
    const ApplySite& st = sites.site[i];
    ps.module[i] = st.module; ps.d1[i] = st.d1; ps.d2[i] = st.d2; ps.Y[i] = st.Y;
    if (!make_map(&sa.xmap[i], st.X, T, st.d1)) return MILORA_E_SHAPE;
    if (!shrink_only && !make_map(&ea.ymap[i], st.Y, T, st.d2)) return MILORA_E_SHAPE;
  }
  for (int i = sites.n; i < kMaxSites; ++i) { sa.xmap[i] = sa.xmap[0]; if (!shrink_only) ea.ymap[i] = ea.ymap[0]; }
  sa.sites = ps; sa.err = ctx->d_err; sa.ws = g->ws_dev; sa.lay = lay; sa.vscratch = ctx->d_vscratch; sa.T = T; sa.rpad = rpad;
  ea.sites = ps; ea.err = ctx->d_err; ea.ws = g->ws_dev; ea.lay = lay; ea.vscratch = ctx->d_vscratch; ea.T = T; ea.rpad = rpad;

  MILORA_CUDA(ctx, cudaFuncSetAttribute(prefill_shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)shrink_smem));
  MILORA_CUDA(ctx, cudaFuncSetAttribute(prefill_expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)expand_smem));
  const size_t grid_s = (size_t)lay.max_tiles * kKSplit, grid_e = (size_t)lay.max_tiles * kNSplit;
  if (grid_s > 0x7fffffffull || grid_e > 0x7fffffffull) return MILORA_E_CAPACITY;
  // Sites that were given the same X (q, k, v; gate, up) and a context that selects several modules per sequence:
  // the shared-input shrink copies every X tile once for all of a sequence's modules among them.
  bool any_shared = false;
  for (int i = 0; i < kMaxSites; ++i) sa.share[i] = i;
  for (int i = 0; i < sites.n; ++i)
    for (int j = 0; j < i; ++j)
      if (sites.site[j].X == sites.site[i].X && sites.site[j].d1 == sites.site[i].d1) {
        sa.share[i] = sa.share[j];
        any_shared = true;
        break;
      }
  sa.K = top_k_of(ctx);
  sa.n_ent = g->n_seq * sa.K;
  sa.stages = kShrinkStages;
  if (any_shared && sa.K > 1) {
    const size_t per = (size_t)kXStage + (size_t)kMaxShare * rpad * 128;
    const size_t two_per_sm = 113 * 1024 - 256, one_per_sm = 220 * 1024 - 256;
    int stages = (int)std::min<size_t>(kShrinkStages, two_per_sm / per);
    if (stages < 4) stages = (int)std::min<size_t>(kShrinkStages, one_per_sm / per);
    if (stages < 2) return MILORA_E_SHAPE;
    sa.stages = stages;
    const size_t smem = (size_t)stages * per + 256;
    MILORA_CUDA(ctx, cudaFuncSetAttribute(prefill_shrink_shared_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MILORA_CUDA(ctx, launch_pdl(prefill_shrink_shared_kernel, dim3((unsigned)grid_s), dim3(kShrinkThreads), smem, s, sa));
  } else {
    MILORA_CUDA(ctx, launch_pdl(prefill_shrink_kernel, dim3((unsigned)grid_s), dim3(kShrinkThreads), shrink_smem, s, sa));
  }
  if (shrink_only) return MILORA_OK;
  MILORA_CUDA(ctx, launch_pdl(prefill_expand_kernel, dim3((unsigned)grid_e), dim3(kExpandThreads), expand_smem, s, ea));
  return MILORA_OK;
}

milora_status launch_apply_prefill_bf16(milora_ctx* ctx, int layer, const ApplySites& sites, const milora_groups* g,
                                        cudaStream_t s) {
  (void)layer;
  return launch_prefill(ctx, sites, g, false, s);
}

// Y = X . W + b with the LoRA term of the routed dense tiles added in the same pass (Eq. 1):
// shrink kernel (partial V) -> pack kernel (V pieces per row block) -> persistent GEMM.
milora_status launch_linear_prefill_bf16(milora_ctx* ctx, int layer, int module, const void* X, const void* Wt,
                                         const void* bias, void* Y, const milora_groups* g, cudaStream_t s) {
  (void)layer;
  if (ctx->desc.dtype != MILORA_BF16) return MILORA_E_SHAPE;
  int d1, d2;
  module_dims(ctx->desc, module, &d1, &d2);
  const int T = g->T;
  const int rpad = (ctx->desc.max_rank + 15) & ~15;
  if (rpad > kLinRPadMax || T < kTileRows || d1 % kLinBK || d2 % kLinBN) return MILORA_E_SHAPE;
  if ((reinterpret_cast<uintptr_t>(X) & 15) || (reinterpret_cast<uintptr_t>(Y) & 15) ||
      (reinterpret_cast<uintptr_t>(Wt) & 15) || (reinterpret_cast<uintptr_t>(bias) & 1))
    return MILORA_E_SHAPE;
  // every check the host can make comes before the first thing is put on the stream
  LinearArgs la;
  if (!make_map(&la.xmap, X, T, d1, kLinBM) || !make_map(&la.wmap, Wt, d2, d1, kLinBN)) return MILORA_E_SHAPE;
  const milora_group_layout_t lay = group_layout(g->n_seq, g->T, top_k_of(ctx));
  const int n_mblk = (T + kLinBM - 1) / kLinBM, n_nblk = d2 / kLinBN;
  const size_t img_bytes = (size_t)kTileRows * rpad * 2;
  const size_t vimg_bytes = (size_t)lay.max_tiles * 2 * img_bytes;
  const size_t cnt_off = (vimg_bytes + 255) & ~size_t(255);
  const size_t job_off = cnt_off + (((size_t)n_mblk * 4 + 255) & ~size_t(255));
  const size_t need = job_off + (size_t)n_mblk * kMaxPieces * 4;
  if (need > ctx->lin_bytes) {
    MILORA_CUDA(ctx, cudaStreamSynchronize(s));
    if (ctx->d_lin) MILORA_CUDA(ctx, cudaFree(ctx->d_lin));
    ctx->d_lin = nullptr;
    ctx->lin_bytes = 0;
    MILORA_CUDA(ctx, cudaMalloc(&ctx->d_lin, need));
    ctx->lin_bytes = need;
  }
  unsigned char* lin = static_cast<unsigned char*>(ctx->d_lin);
  MILORA_CUDA(ctx, cudaMemsetAsync(lin + cnt_off, 0, (size_t)n_mblk * 4, s));

  ApplySites sites;
  sites.n = 1;
  sites.site[0].module = module; sites.site[0].X = X; sites.site[0].Y = nullptr; sites.site[0].d1 = d1; sites.site[0].d2 = d2;
  milora_status st = launch_prefill(ctx, sites, g, true, s);
  if (st != MILORA_OK) return st;

  PackArgs pa;
  pa.err = ctx->d_err; pa.ws = g->ws_dev; pa.lay = lay; pa.vscratch = ctx->d_vscratch; pa.vimg = lin;
  pa.piece_cnt = reinterpret_cast<int32_t*>(lin + cnt_off); pa.piece_job = reinterpret_cast<int32_t*>(lin + job_off);
  pa.module = module; pa.T = T; pa.rpad = rpad; pa.n_mblk = n_mblk;
  if (lay.max_tiles > 0)
    MILORA_CUDA(ctx, launch_pdl(linear_vpack_kernel, dim3((unsigned)lay.max_tiles), dim3(kTileRows), 0, s, pa));

  la.err = ctx->d_err; la.ws = g->ws_dev; la.lay = lay; la.vimg = lin; la.piece_cnt = pa.piece_cnt; la.piece_job = pa.piece_job;
  la.bias = static_cast<const __nv_bfloat16*>(bias); la.Y = static_cast<__nv_bfloat16*>(Y);
  la.T = T; la.d1 = d1; la.d2 = d2; la.rpad = rpad; la.n_mblk = n_mblk; la.n_nblk = n_nblk;
  const size_t smem = (size_t)kLinStages * (kLinAStage + kLinBStage) + (size_t)kTileRows * rpad * 2 + (size_t)rpad * 512 + 256;
  MILORA_CUDA(ctx, cudaFuncSetAttribute(linear_lora_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int grid = std::min(n_mblk * n_nblk, ctx->sm_count);
  MILORA_CUDA(ctx, launch_pdl(linear_lora_kernel, dim3((unsigned)grid), dim3(kLinThreads), smem, s, la));
  return MILORA_OK;
}

}  // namespace milora
