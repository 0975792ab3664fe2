// Token grouping for multi-tenant batches: bucket a step's tokens by (module, tenant) for one layer
// and build the work lists of the apply kernels.
//
// A step is given as sequences of consecutive rows, and the keys of a token depend only on its
// sequence's request slot, so the sort runs over (sequence, selected module) entries (at most kMaxSeq;
// top_k entries per sequence), not over tokens: one CTA per layer sorts the composite keys
// (key << 12 | entry index), which are unique, in shared memory; equal keys then sit next to each other
// in sequence order, which is row order.  Everything after that is prefix sums.  Integer work only; the
// result is the same as a stable sort of the (token, module) pairs by key.
#include <climits>

#include "milora_internal.h"

namespace milora {
namespace {

constexpr int kGMaxThreads = 1024;
constexpr int kSeqBits = 12;  // kMaxSeq = 4096 sequences
static_assert((1 << kSeqBits) == kMaxSeq, "kSeqBits must match kMaxSeq");
constexpr int kSmemArrays = 9;

// Exclusive prefix sums over the block of N ints per thread (scanned together: three barriers in all);
// returns the exclusive values in v, the block totals in total.  wsum holds N x 33 ints.
template <int N>
__device__ inline void block_exscan(int (&v)[N], int (&total)[N], int* wsum) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int inc[N];
#pragma unroll
  for (int k = 0; k < N; ++k) {
    inc[k] = v[k];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, inc[k], o);
      if (lane >= o) inc[k] += t;
    }
  }
  __syncthreads();
  if (lane == 31) {
#pragma unroll
    for (int k = 0; k < N; ++k) wsum[k * 33 + warp] = inc[k];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int k = 0; k < N; ++k) {
      int w = lane < nwarps ? wsum[k * 33 + lane] : 0;
      int winc = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += t;
      }
      wsum[k * 33 + lane] = winc - w;
      if (lane == 31) wsum[k * 33 + 32] = winc;
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < N; ++k) {
    total[k] = wsum[k * 33 + 32];
    v[k] = wsum[k * 33 + warp] + inc[k] - v[k];
  }
}

struct GroupArgs {
  DeviceTables tab;
  const int32_t* cu;        // may be null: every sequence has one row
  const int32_t* seq_slot;
  int32_t* ws;
  size_t ws_stride;
  milora_group_layout_t lay;
  int layer_begin, n_seq, n_ent, n_pad, T;
};

// Shared memory (int32): comp[n_pad], seq_lo[n_pad], seq_len[n_pad], ent_gate[n_pad] (fp32), tok_off[n_pad+1],
// seg_tile[n_pad+1], seg_short[n_pad+1], seg_gather[n_pad+1] (kSmemArrays * n_pad + 8 in total).
__global__ void __launch_bounds__(kGMaxThreads) group_kernel(GroupArgs a) {
  extern __shared__ int32_t sm[];
  __shared__ int wsum[5 * 33];
  const int kGThreads = blockDim.x;
  const int n_pad = a.n_pad, n_seq = a.n_seq;
  int32_t* comp = sm;
  int32_t* seq_lo = comp + n_pad;
  int32_t* seq_len = seq_lo + n_pad;
  float* ent_gate = reinterpret_cast<float*>(seq_len + n_pad);
  int32_t* tok_off = seq_len + 2 * n_pad;
  int32_t* seg_tile = tok_off + n_pad + 1;
  int32_t* seg_short = seg_tile + n_pad + 1;
  int32_t* seg_gather = seg_short + n_pad + 1;
  const int tid = threadIdx.x;
  const int layer = a.layer_begin + blockIdx.x;
  int32_t* ws = a.ws + (size_t)blockIdx.x * a.ws_stride;
  const int max_tenants = a.tab.max_tenants;
  const int K = a.tab.top_k, n_ent = a.n_ent;
  int32_t* seq_tile = ws + a.lay.seq_tile;      // [n_seq][8]: first dense tile per module (-1: none), [7] = module mask
  pdl_launch_dependents();
  pdl_wait();

  // ---- 1. composite keys of the (sequence, selected module) entries, excluded-token count ------
  for (int e = n_ent + tid; e < n_pad; e += kGThreads) comp[e] = INT_MAX;
  int excl = 0;
  for (int i = tid; i < n_seq; i += kGThreads) {
    int lo = i, hi = i + 1;
    const int slot = a.seq_slot[i];          // fetched together with the row range
    if (a.cu) { lo = a.cu[i]; hi = a.cu[i + 1]; }
    bool rows_ok = lo >= 0 && hi >= lo && hi <= a.T;
    if (!rows_ok) atomicOr(a.tab.err, ERR_BAD_ROW);
    int len = rows_ok ? hi - lo : 0;
    seq_lo[i] = lo;
    seq_len[i] = len;
    bool ok = slot >= 0 && slot < a.tab.max_requests;
    if (!ok) atomicOr(a.tab.err, ERR_BAD_SLOT);
    int tenant = -1;
    if (ok && len > 0) tenant = a.tab.slot_tenant[slot];
    const bool tenant_ok = tenant >= 0 && tenant < max_tenants;
    bool any = false;
    int tiled = 0;                             // modules that get dense tiles for this sequence
    for (int j = 0; j < K; ++j) {
      int c = INT_MAX;
      float gt = 1.f;
      if (tenant_ok) {
        const size_t cell = ((size_t)slot * a.tab.n_layers + layer) * K + j;
        const int module = a.tab.route[cell];
        if (module >= 0 && module < MILORA_NMOD) {
          const AdapterEntry& e = a.tab.adapters[adapter_index(tenant, layer, module, a.tab.n_layers)];
          if (e.rank > 0) {
            c = ((module * max_tenants + tenant) << kSeqBits) | (i * K + j);
            any = true;
            if (a.tab.gating) gt = a.tab.gate[cell];
          }
        }
      }
      comp[i * K + j] = c;
      ent_gate[i * K + j] = gt;
      if (c != INT_MAX && len >= kLongSeq) tiled |= 1 << ((c >> kSeqBits) / max_tenants);
    }
    for (int m = 0; m < MILORA_NMOD; ++m) seq_tile[8 * i + m] = -1;
    seq_tile[8 * i + 7] = tiled;
    if (!any) excl += len;
  }
  int n_excl;
  {
    int v1[1] = {excl}, t1[1];
    block_exscan<1>(v1, t1, wsum);
    n_excl = t1[0];
  }

  // ---- 2. sort of the composite keys ---------------------------------------------------------
  if (n_pad <= 256 && n_pad <= kGThreads) {
    // at most one key per thread (a decode batch, a few prompts): rank by counting, three barriers
    // in place of a sorting network.  Valid keys are unique; the padding is ordered by position.
    __syncthreads();
    const int c = tid < n_pad ? comp[tid] : INT_MAX;
    int rank = 0;
    if (tid < n_pad) {
#pragma unroll 8
      for (int j = 0; j < n_pad; ++j) {
        const int o = comp[j];
        rank += (o < c || (o == c && j < tid)) ? 1 : 0;
      }
    }
    __syncthreads();
    if (tid < n_pad) comp[rank] = c;
  } else
  for (int k = 2; k <= n_pad; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      __syncthreads();
      for (int t = tid; t < n_pad / 2; t += kGThreads) {
        int i = 2 * t - (t & (j - 1));      // index with bit j clear
        int l = i + j;
        bool up = (i & k) == 0;
        int x = comp[i], y = comp[l];
        if ((x > y) == up) { comp[i] = y; comp[l] = x; }
      }
    }
  }
  __syncthreads();

  // ---- 3. per-sequence quantities in sorted order; each thread owns consecutive positions ----
  const int per = (n_pad + kGThreads - 1) / kGThreads;
  const int j0 = min(tid * per, n_pad), j1 = min(j0 + per, n_pad);
  int s_tok = 0, s_head = 0, s_tile = 0, s_short = 0, s_act = 0;
  for (int j = j0; j < j1; ++j) {
    int c = comp[j];
    if (c == INT_MAX) break;
    int len = seq_len[(c & (kMaxSeq - 1)) / K];
    s_act += 1;
    s_tok += len;
    s_head += (j == 0 || (comp[j - 1] >> kSeqBits) != (c >> kSeqBits)) ? 1 : 0;
    if (len >= kLongSeq) s_tile += (len + kTileRows - 1) / kTileRows;
    else s_short += len;
  }
  int v5[5] = {s_tok, s_head, s_tile, s_short, s_act}, t5[5];
  block_exscan<5>(v5, t5, wsum);
  int o_tok = v5[0], o_head = v5[1], o_tile = v5[2], o_short = v5[3];
  const int n_active = t5[0], n_seg = t5[1], n_tiles = t5[2], n_short = t5[3], n_act_seq = t5[4];

  TileJob* tiles = reinterpret_cast<TileJob*>(ws + a.lay.tiles);
  int32_t* gather_rows = ws + a.lay.gather_rows;       // row, entry index of every gathered (token, module) pair
  int32_t* seg_key = ws + a.lay.seg_key;
  int32_t* seg_offset = ws + a.lay.seg_offset;
  for (int j = j0; j < j1; ++j) {
    int c = comp[j];
    if (c == INT_MAX) break;
    int key = c >> kSeqBits;
    const int ent = c & (kMaxSeq - 1);
    int lo = seq_lo[ent / K], len = seq_len[ent / K];
    bool head = (j == 0 || (comp[j - 1] >> kSeqBits) != key);
    if (head) {
      seg_key[o_head] = key;
      seg_offset[o_head] = o_tok;
      seg_tile[o_head] = o_tile;
      seg_short[o_head] = o_short;
      ++o_head;
    }
    const int seg = o_head - 1;
    tok_off[j] = o_tok;
    o_tok += len;
    if (len >= kLongSeq) {
      const int module = key / max_tenants;
      const AdapterEntry e = a.tab.adapters[adapter_index(key % max_tenants, layer, module, a.tab.n_layers)];
      TileJob w;
      w.At = e.At; w.B = e.B; w.At_img = e.At_img; w.B_img = e.B_img;
      w.rank = e.rank; w.scale = e.scale * ent_gate[ent]; w.module = module; w.seg = seg; w.rank_pad = e.rank_pad;
      w.ent = ent | (seq_tile[8 * (ent / K) + 7] << 16);
      seq_tile[8 * (ent / K) + module] = o_tile;
      for (int r = 0; r < len; r += kTileRows) {
        w.start = lo + r;
        w.count = min(kTileRows, len - r);
        tiles[o_tile++] = w;
      }
    } else {
      for (int r = 0; r < len; ++r) {
        gather_rows[2 * o_short] = lo + r;
        gather_rows[2 * o_short + 1] = ent;
        ++o_short;
      }
    }
  }
  if (tid == 0) {
    seg_offset[n_seg] = n_active;
    seg_tile[n_seg] = n_tiles;
    seg_short[n_seg] = n_short;
    tok_off[n_act_seq] = n_active;
  }
  __syncthreads();

  // ---- 4. perm: token q of the sorted order ------------------------------------------------
  int32_t* perm = ws + a.lay.perm;
  // one warp per sorted sequence: its rows are consecutive, so the writes are coalesced
  for (int j = tid >> 5; j < n_act_seq; j += kGThreads / 32) {
    const int i = (comp[j] & (kMaxSeq - 1)) / K;
    const int lo = seq_lo[i], len = seq_len[i], off = tok_off[j];
    for (int t = tid & 31; t < len; t += 32) perm[off + t] = lo + t;
  }

  // ---- 5. gather jobs: chunks of kGatherRows short rows per segment ---------------------------
  const int sper = (n_seg + kGThreads - 1) / kGThreads;
  const int s0 = min(tid * sper, n_seg), s1 = min(s0 + sper, n_seg);
  int g_cnt = 0;
  for (int s = s0; s < s1; ++s) g_cnt += (seg_short[s + 1] - seg_short[s] + kGatherRows - 1) / kGatherRows;
  int n_gather, o_g;
  {
    int v1[1] = {g_cnt}, t1[1];
    block_exscan<1>(v1, t1, wsum);
    o_g = v1[0];
    n_gather = t1[0];
  }
  GatherJob* gather = reinterpret_cast<GatherJob*>(ws + a.lay.gather);
  for (int s = s0; s < s1; ++s) {
    seg_gather[s] = o_g;
    const int b = seg_short[s], e = seg_short[s + 1];
    if (b == e) continue;
    const int key = seg_key[s];
    const int module = key / max_tenants;
    const AdapterEntry ent = a.tab.adapters[adapter_index(key % max_tenants, layer, module, a.tab.n_layers)];
    GatherJob w;
    w.At = ent.At; w.B = ent.B; w.rank = ent.rank; w.scale = ent.scale; w.module = module;
    for (int r = b; r < e; r += kGatherRows) {
      w.count = min(kGatherRows, e - r);
#pragma unroll
      for (int t = 0; t < kGatherRows; ++t) {
        w.rows[t] = (t < w.count) ? gather_rows[2 * (r + t)] : -1;
        w.gate[t] = (t < w.count) ? ent_gate[gather_rows[2 * (r + t) + 1]] : 0.f;
      }
      gather[o_g++] = w;
    }
  }
  if (tid == 0) seg_gather[n_seg] = n_gather;
  __syncthreads();

  // ---- 6. header and per-module ranges -----------------------------------------------------
  if (tid < 8) {
    // first segment whose module is >= tid
    int lo = 0, hi = n_seg;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (seg_key[mid] / max_tenants < tid) lo = mid + 1; else hi = mid;
    }
    ws[a.lay.mod_offset + tid] = lo;
    ws[a.lay.mod_tile_offset + tid] = seg_tile[lo];
    ws[a.lay.mod_gather_offset + tid] = seg_gather[lo];
  }
  if (tid < kHeaderInts) {
    int v = 0;
    if (tid == H_NSEG) v = n_seg;
    else if (tid == H_NEXCL) v = n_excl;
    else if (tid == H_NACTIVE) v = n_active;
    else if (tid == H_NTILES) v = n_tiles;
    else if (tid == H_NGATHER) v = n_gather;
    ws[a.lay.header + tid] = v;
  }
}

}  // namespace

milora_status launch_group(milora_ctx* ctx, int layer_begin, int n_layers, const int32_t* cu, const int32_t* seq_slot,
                           int n_seq, int T, int32_t* ws, size_t ws_stride, cudaStream_t s) {
  if ((long long)ctx->desc.max_tenants * MILORA_NMOD >= (1ll << (31 - kSeqBits))) return MILORA_E_CAPACITY;
  GroupArgs a;
  a.tab = device_tables(ctx);
  a.cu = cu; a.seq_slot = seq_slot; a.ws = ws; a.ws_stride = ws_stride;
  a.lay = group_layout(n_seq, T, top_k_of(ctx));
  a.layer_begin = layer_begin; a.n_seq = n_seq; a.T = T;
  a.n_ent = n_seq * top_k_of(ctx);
  int n_pad = 2;
  while (n_pad < a.n_ent) n_pad <<= 1;
  a.n_pad = n_pad;
  size_t smem = ((size_t)n_pad * kSmemArrays + 8) * sizeof(int32_t);
  if (smem > 48 * 1024) {
    MILORA_CUDA(ctx, cudaFuncSetAttribute(group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  }
  // few sequences (a decode batch): a smaller block makes every barrier and scan cheaper; many rows (prompts): perm is
  // written by one warp per sequence, 32 rows per pass, and wants warps (32,768 rows: 3.9 us with 4 warps, 1 with 16)
  int threads = std::max(128, std::min(kGMaxThreads, n_pad));
  threads = std::max(threads, std::min(kGMaxThreads, (T / 64) & ~31));
  MILORA_CUDA(ctx, launch_pdl(group_kernel, dim3(n_layers), dim3(threads), smem, s, a));
  return MILORA_OK;
}

}  // namespace milora
