// Importance (Eq. 6) and Top-K channel / layer selection in the three modes of Table 2.
//
// Keys are fp32 means accumulated in fp64.  Ranking: larger key first, equal keys by
// smaller index; winners are emitted in ascending index order.  Top-K is a radix select on
// the order-preserving integer image of the key (4 passes of 8 bits) followed by an
// order-preserving compaction, one block per ranked segment.
#include "internal.h"

namespace efqat {

struct LayerEntry {
  const float* W;
  int N, K;
  int row_off;   // first global channel id of the layer
  int k;         // CWPL: channels kept in this layer
  int out_off;   // CWPL: position of the layer's first index in idx
  int pad;
};
static_assert(sizeof(LayerEntry) == 32, "LayerEntry layout");

static const int TABLE_CHUNK = 96;
struct TableChunk {
  LayerEntry e[TABLE_CHUNK];
};

__global__ void table_write_kernel(TableChunk chunk, int count, LayerEntry* __restrict__ dst) {
  pdl_trigger();
  pdl_wait();
  const int i = threadIdx.x;
  if (i < count) dst[i] = chunk.e[i];
}

__device__ __forceinline__ int layer_of_row(const LayerEntry* __restrict__ table, int L, int row) {
  int lo = 0, hi = L - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (table[mid].row_off <= row) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ double abs4(const float4 a) {
  return (static_cast<double>(fabsf(a.x)) + static_cast<double>(fabsf(a.y))) +
         (static_cast<double>(fabsf(a.z)) + static_cast<double>(fabsf(a.w)));
}

// One warp per output channel: sum |w| over the row in fp64, key = fl32(sum / K).
__global__ void __launch_bounds__(256) row_importance_kernel(const LayerEntry* __restrict__ table, int L,
                                                             int total_rows, float* __restrict__ keys,
                                                             double* __restrict__ rowsum) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int row = blockIdx.x * warps_per_block + (threadIdx.x >> 5); row < total_rows;
       row += gridDim.x * warps_per_block) {
    const int l = layer_of_row(table, L, row);
    const LayerEntry e = table[l];
    const float* w = e.W + static_cast<int64_t>(row - e.row_off) * e.K;
    double acc = 0.0;
    if ((e.K & 3) == 0 && (reinterpret_cast<uintptr_t>(w) & 15) == 0) {
      const float4* w4 = reinterpret_cast<const float4*>(w);
      const int n4 = e.K >> 2;
      int i = lane;
      for (; i + 224 < n4; i += 256) {    // eight independent 16-byte loads in flight per lane
        float4 t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = __ldg(w4 + i + 32 * u);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc += abs4(t[u]);
      }
      for (; i + 96 < n4; i += 128) {     // four
        const float4 a = __ldg(w4 + i), b = __ldg(w4 + i + 32), c = __ldg(w4 + i + 64), d = __ldg(w4 + i + 96);
        acc += abs4(a);
        acc += abs4(b);
        acc += abs4(c);
        acc += abs4(d);
      }
      for (; i < n4; i += 32) acc += abs4(__ldg(w4 + i));
    } else {
      for (int i = lane; i < e.K; i += 32) acc += static_cast<double>(fabsf(w[i]));
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      rowsum[row] = acc;
      keys[row] = static_cast<float>(acc / static_cast<double>(e.K));
    }
  }
}

// LWPN: key of a layer = mean |w| over all of its weights.
__global__ void __launch_bounds__(256) layer_importance_kernel(const LayerEntry* __restrict__ table,
                                                               const double* __restrict__ rowsum,
                                                               float* __restrict__ layer_keys) {
  pdl_trigger();
  pdl_wait();
  const LayerEntry e = table[blockIdx.x];
  double acc = 0.0;
  for (int i = threadIdx.x; i < e.N; i += blockDim.x) acc += rowsum[e.row_off + i];
  __shared__ double sh[256];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0)
    layer_keys[blockIdx.x] = static_cast<float>(sh[0] / (static_cast<double>(e.N) * static_cast<double>(e.K)));
}

// Order-preserving map float -> uint32 (larger float <-> larger integer).
__device__ __forceinline__ uint32_t key_bits(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

static const int TOPK_THREADS = 1024;
static const int TOPK_SMEM_KEYS = 8192;

// Block-wide exclusive scan of two counters (all TOPK_THREADS threads must call).
__device__ __forceinline__ void block_scan2(int a, int b, int& pa, int& pb, int* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int ua = __shfl_up_sync(0xffffffffu, ia, o), ub = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ua; ib += ub; }
  }
  if (lane == 31) { sh[warp] = ia; sh[32 + warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    const int wa = sh[lane], wb = sh[32 + lane];
    int sa = wa, sb = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int ua = __shfl_up_sync(0xffffffffu, sa, o), ub = __shfl_up_sync(0xffffffffu, sb, o);
      if (lane >= o) { sa += ua; sb += ub; }
    }
    sh[lane] = sa - wa;
    sh[32 + lane] = sb - wb;
  }
  __syncthreads();
  pa = sh[warp] + ia - a;
  pb = sh[32 + warp] + ib - b;
  __syncthreads();
}

// One block per segment.  table != null: segment = layer blockIdx.x (CWPL).  table == null:
// the single segment [0, single_len) with budget single_k.
__global__ void __launch_bounds__(TOPK_THREADS) topk_kernel(const float* __restrict__ keys,
                                                            const LayerEntry* __restrict__ table, int single_len,
                                                            int single_k, int32_t* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  __shared__ int hist[256];
  __shared__ int suf[257];
  __shared__ int scan_sh[64];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  __shared__ uint32_t skeys[TOPK_SMEM_KEYS];

  int begin = 0, n = single_len, k = single_k, out_off = 0;
  if (table) {
    const LayerEntry e = table[blockIdx.x];
    begin = e.row_off; n = e.N; k = e.k; out_off = e.out_off;
  }
  if (k <= 0 || n <= 0) return;     // uniform over the block
  if (k > n) k = n;
  const float* kp = keys + begin;
  int32_t* op = out + out_off;

  // Segments of up to TOPK_SMEM_KEYS keys are read from global memory once, as their
  // order-preserving integer images, and every pass works on the shared copy.
  const bool cached = n <= TOPK_SMEM_KEYS;
  if (cached) {
    for (int i = threadIdx.x; i < n; i += blockDim.x) skeys[i] = key_bits(kp[i]);
    __syncthreads();
  }
  auto key_at = [&](int i) { return cached ? skeys[i] : key_bits(kp[i]); };

  uint32_t prefix = 0, mask = 0;
  int remaining = k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int base = 0; base < n; base += blockDim.x) {
      const int i = base + threadIdx.x;
      int digit = -1;                                // -1: not a candidate any more
      if (i < n) {
        const uint32_t kb = key_at(i);
        if ((kb & mask) == prefix) digit = (kb >> shift) & 255;
      }
      // Importance keys share their leading bytes, so in the first passes a whole warp usually
      // lands in one bin: that case costs one atomic per warp, the general one one per lane.
      const uint32_t cand = __ballot_sync(0xffffffffu, digit >= 0);
      if (cand) {
        const int leader = __ffs(cand) - 1;
        const int d0 = __shfl_sync(0xffffffffu, digit, leader);
        const bool same = __all_sync(0xffffffffu, digit < 0 || digit == d0);
        if (same) {
          if ((threadIdx.x & 31) == leader) atomicAdd(&hist[d0], __popc(cand));
        } else if (digit >= 0) {
          atomicAdd(&hist[digit], 1);
        }
      }
    }
    __syncthreads();
    // digit of the k-th largest candidate: largest d whose suffix count reaches `remaining`.
    // Suffix sums over the 256 bins: inclusive suffix inside each of 8 warps by shuffles,
    // then the totals of the warps above are added.
    {
      const int d = threadIdx.x, lane = d & 31, warp = d >> 5;
      int v = (d < 256) ? hist[d] : 0;
      if (d < 256) {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int u = __shfl_down_sync(0xffffffffu, v, o);
          if (lane + o < 32) v += u;
        }
        if (lane == 0) scan_sh[warp] = v;          // total of this warp's 32 bins
      }
      __syncthreads();
      if (d < 256) {
        int above = 0;
        for (int w2 = warp + 1; w2 < 8; ++w2) above += scan_sh[w2];
        suf[d] = v + above;
      }
      if (d == 0) suf[256] = 0;
      __syncthreads();
      if (d < 256 && ((suf[d] >= remaining && suf[d + 1] < remaining) || (d == 0 && suf[0] < remaining))) {
        sh_prefix = prefix | (static_cast<uint32_t>(d) << shift);
        sh_remaining = remaining - suf[d + 1];
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    remaining = sh_remaining;
    mask |= 255u << shift;
    __syncthreads();
  }
  // prefix = image of the k-th largest key; `remaining` of the keys equal to it are taken,
  // those with the smallest indices.  Each thread owns a contiguous index range.
  const uint32_t thr = prefix;
  const int per = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min(n, static_cast<int>(threadIdx.x) * per), hi = min(n, lo + per);
  int gt = 0, eq = 0;
  for (int i = lo; i < hi; ++i) {
    const uint32_t kb = key_at(i);
    gt += kb > thr;
    eq += kb == thr;
  }
  int pg, pe;
  block_scan2(gt, eq, pg, pe, scan_sh);
  int pos = pg + min(pe, remaining);
  int erank = pe;
  for (int i = lo; i < hi; ++i) {
    const uint32_t kb = key_at(i);
    bool take = kb > thr;
    if (kb == thr) {
      take = erank < remaining;
      ++erank;
    }
    if (take) op[pos++] = i;
  }
}

// ---- Top-K of one large segment (per-network ranking) spread over many blocks ------------
// Same radix select, but every pass is a grid-wide histogram followed by a one-block digit
// pick, and the order-preserving compaction uses per-block counts and a scan over them.
struct TopkState {
  uint32_t prefix, mask;
  int remaining, pad;
};
static const int BIG_CHUNK = 4096;      // keys per block in the count / write kernels

__global__ void topk_big_init_kernel(TopkState* st, int k, int* ghist) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x < 256) ghist[threadIdx.x] = 0;
  if (threadIdx.x == 0) {
    st->prefix = 0; st->mask = 0; st->remaining = k; st->pad = 0;
  }
}
__global__ void __launch_bounds__(256) topk_big_hist_kernel(const float* __restrict__ keys, int n,
                                                            const TopkState* __restrict__ st, int shift,
                                                            int* __restrict__ ghist) {
  pdl_trigger();
  pdl_wait();
  __shared__ int sh[256];
  sh[threadIdx.x] = 0;
  __syncthreads();
  const uint32_t prefix = st->prefix, mask = st->mask;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint32_t kb = key_bits(keys[i]);
    if ((kb & mask) == prefix) atomicAdd(&sh[(kb >> shift) & 255], 1);
  }
  __syncthreads();
  if (sh[threadIdx.x]) atomicAdd(&ghist[threadIdx.x], sh[threadIdx.x]);
}
__global__ void __launch_bounds__(256) topk_big_pick_kernel(TopkState* st, int shift, int* ghist) {
  pdl_trigger();
  pdl_wait();
  __shared__ int suf[257];
  const int d = threadIdx.x;
  suf[d] = ghist[d];
  if (d == 0) suf[256] = 0;
  __syncthreads();
  // inclusive suffix sums: suf[d] = number of candidate keys whose digit is >= d
  for (int o = 1; o < 256; o <<= 1) {
    const int v = (d + o < 256) ? suf[d + o] : 0;
    __syncthreads();
    suf[d] += v;
    __syncthreads();
  }
  const int remaining = st->remaining;
  __syncthreads();
  const bool mine = suf[d] >= remaining && suf[d + 1] < remaining;
  if (mine || (d == 0 && suf[0] < remaining)) {
    st->prefix |= static_cast<uint32_t>(d) << shift;
    st->mask |= 255u << shift;
    st->remaining = remaining - suf[d + 1];
  }
  ghist[d] = 0;
}
__global__ void __launch_bounds__(TOPK_THREADS) topk_big_count_kernel(const float* __restrict__ keys, int n,
                                                                      const TopkState* __restrict__ st,
                                                                      int* __restrict__ counts) {
  pdl_trigger();
  pdl_wait();
  __shared__ int red[2][32];
  const uint32_t thr = st->prefix;
  const int lo = blockIdx.x * BIG_CHUNK, hi = min(n, lo + BIG_CHUNK);
  int gt = 0, eq = 0;
  for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    const uint32_t kb = key_bits(keys[i]);
    gt += kb > thr;
    eq += kb == thr;
  }
  for (int o = 16; o > 0; o >>= 1) {
    gt += __shfl_xor_sync(0xffffffffu, gt, o);
    eq += __shfl_xor_sync(0xffffffffu, eq, o);
  }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = gt; red[1][threadIdx.x >> 5] = eq; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int a = 0, b = 0;
    for (int w = 0; w < 32; ++w) { a += red[0][w]; b += red[1][w]; }
    counts[2 * blockIdx.x] = a;
    counts[2 * blockIdx.x + 1] = b;
  }
}
__global__ void topk_big_scan_kernel(const int* __restrict__ counts, int blocks, int* __restrict__ offs) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int a = 0, b = 0;
  for (int i = 0; i < blocks; ++i) {
    offs[2 * i] = a;
    offs[2 * i + 1] = b;
    a += counts[2 * i];
    b += counts[2 * i + 1];
  }
}
__global__ void __launch_bounds__(TOPK_THREADS) topk_big_write_kernel(const float* __restrict__ keys, int n,
                                                                      const TopkState* __restrict__ st,
                                                                      const int* __restrict__ offs,
                                                                      int32_t* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  __shared__ int scan_sh[64];
  __shared__ int carry[2];
  const uint32_t thr = st->prefix;
  const int R = st->remaining;
  const int lo = blockIdx.x * BIG_CHUNK, hi = min(n, lo + BIG_CHUNK);
  if (threadIdx.x == 0) { carry[0] = offs[2 * blockIdx.x]; carry[1] = offs[2 * blockIdx.x + 1]; }
  __syncthreads();
  for (int base = lo; base < hi; base += blockDim.x) {
    const int i = base + threadIdx.x;
    int gt = 0, eq = 0;
    if (i < hi) {
      const uint32_t kb = key_bits(keys[i]);
      gt = kb > thr;
      eq = kb == thr;
    }
    int pg, pe;
    block_scan2(gt, eq, pg, pe, scan_sh);
    const int g_before = carry[0] + pg, e_before = carry[1] + pe;
    if (gt || (eq && e_before < R)) out[g_before + min(e_before, R)] = i;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) { carry[0] = g_before + gt; carry[1] = e_before + eq; }
    __syncthreads();
  }
}

__global__ void cwpl_offsets_kernel(const LayerEntry* __restrict__ table, int L, int total,
                                    int32_t* __restrict__ offsets) {
  pdl_trigger();
  pdl_wait();
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l < L) offsets[l] = table[l].out_off;
  if (l == L) offsets[L] = total;
}

// CWPN: sel holds the k_tot winning global ids in ascending order.
__global__ void cwpn_split_kernel(const LayerEntry* __restrict__ table, int L, const int32_t* __restrict__ sel,
                                  int k_tot, int32_t* __restrict__ idx, int32_t* __restrict__ offsets) {
  pdl_trigger();
  pdl_wait();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < k_tot) {
    const int g = sel[j];
    idx[j] = g - table[layer_of_row(table, L, g)].row_off;
  }
  if (j <= L) {
    // offsets[l] = number of winners with global id < row_off[l]
    const int bound = (j < L) ? table[j].row_off : INT32_MAX;
    int lo = 0, hi = k_tot;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (sel[mid] < bound) lo = mid + 1; else hi = mid;
    }
    offsets[j] = lo;
  }
}

// LWPN: lsel holds the k_L winning layer ids ascending; offsets = prefix of N_l over kept layers.
__global__ void lwpn_offsets_kernel(const LayerEntry* __restrict__ table, int L, const int32_t* __restrict__ lsel,
                                    int k_L, int32_t* __restrict__ keep, int32_t* __restrict__ offsets) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int p = 0, off = 0;
  for (int l = 0; l < L; ++l) {
    const bool kept = (p < k_L && lsel[p] == l);
    if (kept) ++p;
    keep[l] = kept;
    offsets[l] = off;
    if (kept) off += table[l].N;
  }
  offsets[L] = off;
}
__global__ void lwpn_fill_kernel(const LayerEntry* __restrict__ table, int L, int total_rows,
                                 const int32_t* __restrict__ keep, const int32_t* __restrict__ offsets,
                                 int32_t* __restrict__ idx) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= total_rows) return;
  const int l = layer_of_row(table, L, row);
  if (keep[l]) idx[offsets[l] + (row - table[l].row_off)] = row - table[l].row_off;
}

// ------------------------------------------------------------------ host side
struct SelectWs {
  LayerEntry* table;
  double* rowsum;
  float* keys;
  int32_t* sel;
  float* layer_keys;
  int32_t* lsel;
  int32_t* keep;
  TopkState* big_state;
  int* big_hist;
  int* big_counts;
  int* big_offs;
  size_t bytes;
};

static SelectWs carve(void* ws, int L, int64_t total) {
  SelectWs w;
  char* p = static_cast<char*>(ws);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* r = p ? p + off : nullptr;
    off += static_cast<size_t>(round_up(static_cast<int64_t>(bytes), 256));
    return r;
  };
  w.table = reinterpret_cast<LayerEntry*>(take(sizeof(LayerEntry) * static_cast<size_t>(L)));
  w.rowsum = reinterpret_cast<double*>(take(sizeof(double) * static_cast<size_t>(total)));
  w.keys = reinterpret_cast<float*>(take(sizeof(float) * static_cast<size_t>(total)));
  w.sel = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * static_cast<size_t>(total)));
  w.layer_keys = reinterpret_cast<float*>(take(sizeof(float) * static_cast<size_t>(L)));
  w.lsel = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * static_cast<size_t>(L)));
  w.keep = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * static_cast<size_t>(L)));
  const size_t big_blocks = static_cast<size_t>(ceil_div(total, BIG_CHUNK));
  w.big_state = reinterpret_cast<TopkState*>(take(sizeof(TopkState)));
  w.big_hist = reinterpret_cast<int*>(take(256 * sizeof(int)));
  w.big_counts = reinterpret_cast<int*>(take(2 * big_blocks * sizeof(int)));
  w.big_offs = reinterpret_cast<int*>(take(2 * big_blocks * sizeof(int)));
  w.bytes = off;
  return w;
}

size_t select_workspace_bytes(int L, int64_t total_channels) { return carve(nullptr, L, total_channels).bytes; }

int run_select(int mode, int L, const efqat_layer_desc* layers, const float* const* weights, const int64_t* k,
               int32_t* idx, int32_t* offsets, float* importance, void* ws, size_t ws_bytes, int* status,
               cudaStream_t st) {
  (void)status;
  int64_t total = 0;
  for (int l = 0; l < L; ++l) {
    if (layers[l].N < 1 || layers[l].K < 1) return EFQAT_ERR_SHAPE;
    if (!weights[l]) return EFQAT_ERR_NULL;
    total += layers[l].N;
  }
  if (total > INT32_MAX) return EFQAT_ERR_SHAPE;
  if (mode == EFQAT_CWPL) {
    for (int l = 0; l < L; ++l)
      if (k[l] < 0 || k[l] > layers[l].N) return EFQAT_ERR_K_RANGE;
  } else if (mode == EFQAT_CWPN) {
    if (k[0] < 0 || k[0] > total) return EFQAT_ERR_K_RANGE;
  } else if (mode == EFQAT_LWPN) {
    if (k[0] < 0 || k[0] > L) return EFQAT_ERR_K_RANGE;
  } else {
    return EFQAT_ERR_MODE;
  }
  const SelectWs w = carve(ws, L, total);
  if (!ws || ws_bytes < w.bytes) return EFQAT_ERR_WORKSPACE;

  // layer table -> device, passed through kernel parameters (no host staging buffer)
  int64_t row_off = 0, out_off = 0;
  for (int base = 0; base < L; base += TABLE_CHUNK) {
    TableChunk chunk;
    const int cnt = (L - base < TABLE_CHUNK) ? L - base : TABLE_CHUNK;
    for (int i = 0; i < cnt; ++i) {
      const int l = base + i;
      LayerEntry e;
      e.W = weights[l];
      e.N = static_cast<int>(layers[l].N);
      e.K = static_cast<int>(layers[l].K);
      e.row_off = static_cast<int>(row_off);
      e.k = (mode == EFQAT_CWPL) ? static_cast<int>(k[l]) : 0;
      e.out_off = static_cast<int>(out_off);
      e.pad = 0;
      chunk.e[i] = e;
      row_off += layers[l].N;
      out_off += e.k;
    }
    count_launches(1);
    launch_dependent(table_write_kernel, 1, TABLE_CHUNK, 0, st, 1, chunk, cnt, w.table + base);
  }
  const int tot = static_cast<int>(total);
  {
    int64_t blocks = ceil_div(total, 8);
    if (blocks > 148 * 8) blocks = 148 * 8;
    count_launches(1);
    launch_dependent(row_importance_kernel, static_cast<unsigned>(blocks), 256, 0, st, 1, w.table, L, tot, w.keys, w.rowsum);
  }
  if (mode == EFQAT_CWPL) {
    count_launches(2);
    launch_dependent(topk_kernel, L, TOPK_THREADS, 0, st, 1, w.keys, w.table, 0, 0, idx);
    launch_dependent(cwpl_offsets_kernel, static_cast<unsigned>(ceil_div(L + 1, 256)), 256, 0, st, 1, w.table, L,
                                                                                    static_cast<int>(out_off),
                                                                                    offsets);
    if (importance) cudaMemcpyAsync(importance, w.keys, sizeof(float) * total, cudaMemcpyDeviceToDevice, st);
  } else if (mode == EFQAT_CWPN) {
    const int kt = static_cast<int>(k[0]);
    if (tot > 4 * BIG_CHUNK && kt > 0) {
      const int blocks = static_cast<int>(ceil_div(tot, BIG_CHUNK));
      int hgrid = static_cast<int>(ceil_div(tot, 256 * 4));
      if (hgrid > 148 * 4) hgrid = 148 * 4;
      count_launches(13);
      launch_dependent(topk_big_init_kernel, 1, 256, 0, st, 1, w.big_state, kt, w.big_hist);
      for (int shift = 24; shift >= 0; shift -= 8) {
        launch_dependent(topk_big_hist_kernel, hgrid, 256, 0, st, 1, w.keys, tot, w.big_state, shift, w.big_hist);
        launch_dependent(topk_big_pick_kernel, 1, 256, 0, st, 1, w.big_state, shift, w.big_hist);
      }
      launch_dependent(topk_big_count_kernel, blocks, TOPK_THREADS, 0, st, 1, w.keys, tot, w.big_state, w.big_counts);
      launch_dependent(topk_big_scan_kernel, 1, 32, 0, st, 1, w.big_counts, blocks, w.big_offs);
      launch_dependent(topk_big_write_kernel, blocks, TOPK_THREADS, 0, st, 1, w.keys, tot, w.big_state, w.big_offs, w.sel);
    } else {
      count_launches(1);
      launch_dependent(topk_kernel, 1, TOPK_THREADS, 0, st, 1, w.keys, nullptr, tot, kt, w.sel);
    }
    count_launches(1);
    const int work = (kt > L + 1) ? kt : L + 1;
    launch_dependent(cwpn_split_kernel, static_cast<unsigned>(ceil_div(work, 256)), 256, 0, st, 1, w.table, L, w.sel, kt, idx,
                                                                                 offsets);
    if (importance) cudaMemcpyAsync(importance, w.keys, sizeof(float) * total, cudaMemcpyDeviceToDevice, st);
  } else {
    const int kl = static_cast<int>(k[0]);
    count_launches(4);
    launch_dependent(layer_importance_kernel, L, 256, 0, st, 1, w.table, w.rowsum, w.layer_keys);
    launch_dependent(topk_kernel, 1, TOPK_THREADS, 0, st, 1, w.layer_keys, nullptr, L, kl, w.lsel);
    launch_dependent(lwpn_offsets_kernel, 1, 32, 0, st, 1, w.table, L, w.lsel, kl, w.keep, offsets);
    launch_dependent(lwpn_fill_kernel, static_cast<unsigned>(ceil_div(total, 256)), 256, 0, st, 1, w.table, L, tot, w.keep, offsets,
                                                                                 idx);
    if (importance) cudaMemcpyAsync(importance, w.layer_keys, sizeof(float) * L, cudaMemcpyDeviceToDevice, st);
  }
  return (cudaGetLastError() == cudaSuccess) ? EFQAT_OK : EFQAT_ERR_CUDA;
}

}  // namespace efqat
