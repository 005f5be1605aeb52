// bf16 x bf16 -> fp32 GEMM core on the 5th-generation tensor cores (tcgen05 / TMEM),
// operands staged by TMA into 128-byte-swizzled shared memory, with three fused epilogues:
//   EPI_FWD : Y = s_x * s_w[n] * acc + bias[n]                         (forward, Section 3.1)
//   EPI_DX  : dX = acc * [x not clipped]; partial sums of dS_x, dZ_x   (Eq. 5 + STE)
//   EPI_PART: fp32 partial products of the (partial) weight gradient   (Algorithm 1)
//
// Persistent kernel, one CTA per SM, looping over 128 x BN output tiles:
//   warp 0  lane 0 : TMA producer over a ring of shared-memory stages
//   warp 1  lane 0 : issues tcgen05.mma into one of two TMEM accumulators; warp 1 owns TMEM
//   warps 2..5     : epilogue of the previous tile, overlapped with the next tile's main loop;
//                    each warp reads its 32-lane quarter of the accumulator, fetches its slice
//                    of X with TMA (EPI_DX) and writes its slice of the output with TMA stores
//                    from a swizzled staging buffer, so global traffic is in whole 128-byte rows
// With CTA2 = 1 two CTAs of a cluster work as a pair on a 256 x BN tile (tcgen05 cta_group::2):
// each CTA stages its own 128 rows of A and one half of the B tile, the leader CTA issues the
// MMAs for both, and every CTA runs the epilogue of its own 128 rows.  This halves the B
// traffic from L2 per FLOP, which is what bounds the one-CTA tiles.  No TMA multicast is used.
// Either operand may be stored with the contraction dimension contiguous ("K-major") or
// with the other dimension contiguous ("MN-major"); the shared-memory and instruction
// descriptors carry the difference, so no transposed copies are ever made.
#include "internal.h"
#include "ptx.cuh"

namespace efqat {

using namespace ptx;

static const int BM = 128;          // tile rows = UMMA M = TMEM lanes
static const int BK = 64;           // contraction elements per stage (one 128-byte swizzle row)
static const int UMMA_K = 16;
static const int MAX_STAGES = 8;
static const int A_STAGE_BYTES = BM * BK * 2;   // 16 KiB
static const int CHUNK_BYTES = 64 * BK * 2;     // one 64-wide MN-major chunk, 8 KiB
static const int EPI_WARPS = 8;
static const int GEMM_THREADS = 64 + 32 * EPI_WARPS;
static const int ACC_STRIDE = 256;              // TMEM columns between the two accumulators
static const int TMEM_COLS = 512;
static const int HB_BYTES = 32 * 64;            // staging block of one epilogue warp: 32 rows x 64 B
static const int MAX_TAPS = 49;                // filter taps of one launch (7 x 7)
static const double L2_PANEL_BYTES = 32.0 * 1024 * 1024;   // operand slice kept resident in L2 by the tile order

// Convolution geometry as the kernel needs it (mode 0 = plain matrices).
struct ConvP {
  int mode;                 // 1 forward, 2 grad-input, 3 grad-weight
  int tw, th, tb;           // pixel box: one 128-row tile (modes 1, 2) or one 64-row contraction block (mode 3)
  int tiles_w, tiles_h;     // boxes along W and H (boxes along B follow from the tile / block count)
  int dimH, dimB;           // extent of the tiled pixel space in H and B (store / load guards)
  int C;                    // channels of the 4-D A tensor (Cin for modes 1 and 3, N for mode 2)
  int cchunks;              // 64-channel chunks of C (the last one zero-filled past C by the TMA unit)
  int wcols;                // columns of one filter tap in the weight matrix (= Cin)
  // Filter taps of this launch.  Tap t reads the A tensor through map tap_map[t] (strided
  // convolutions see the input as stride x stride interleaved sub-grids, one tensor map each)
  // with its pixel box shifted by (tap_dw[t], tap_dh[t]); tap_rs[t] = r * S + s is its position
  // in the filter.  Grad-input launches carry only the taps that reach their pixel class.
  int ntaps;
  int8_t tap_dh[MAX_TAPS], tap_dw[MAX_TAPS];
  uint8_t tap_map[MAX_TAPS], tap_rs[MAX_TAPS];
};

struct GemmParams {
  ConvP cv;
  int64_t Mr, Nc;
  int nkb;            // number of BK blocks along the contraction
  int BN;             // tile columns (multiple of 16, <= 256)
  int stages;
  int i8;             // EPI_FWD on 8-bit integer operands (kind::i8): 128 contraction elements per k-block
  int bk;             // contraction elements per k-block: 64 (bf16) or 128 (8-bit)
  int a_signed;       // i8: activation codes are signed (symmetric quantizer)
  const int32_t* wsum;
  int kps;            // k-blocks per stage: one barrier round trip covers kps * 64 contraction elements
  int merged;         // MN-major operands arrive as one TMA box per 64-wide chunk and stage (plain matrices only)
  int b_stage_bytes;
  // One stage of the ring = a_region_bytes of A operand + b_region_bytes of B operand; k-block u of
  // the stage has its A operand a_sub_off * u bytes into the A region.
  int a_region_bytes, b_region_bytes, a_sub_off;
  // Convolutions whose taps form a grid (filter rows x filter columns, consecutive row shifts):
  // the taps of one filter column differ only by a shift of whole pixel rows, so ONE box of
  // th + colshare - 1 pixel rows serves all `colshare` of them (each tap's operand starts
  // tw pixels = tw * 128 bytes further on, a multiple of the 1024-byte swizzle atom because tw is a
  // multiple of 8).  0: every tap loads a box of its own.  a_tx: bytes of that shared box.
  int colshare, a_tx;
  // The whole B operand (all taps and channel chunks) stays in shared memory for the life of the
  // CTA: nkb blocks of b_stage_bytes behind the ring (tiles_n == 1 only).
  int bres;
  int splits;
  int tiles_m, tiles_n;
  int panel_dir, panel;   // order of the tiles in the work list (see tile_coords)
  int hint_a, hint_b;     // L2 eviction policy of the A / B operand loads (plain matrices): see ptx::l2_policy
  int blk_cols;       // output columns per 64-byte staging row: 32 (bf16) or 16 (fp32)
  int out_bufs;       // staging buffers per epilogue warp (2 when shared memory allows)
  const float* col_scale;
  const float* col_bias;
  const float* s_x; const float* z_x; int x_bits, x_sym;
  float* partials;    // EPI_DX: [tile][quarter][2]
  float* out;         // EPI_PART
  int64_t ldo;
  int64_t split_stride;
  int64_t part_cols;
  int* status;
  int defer_wait;
};

struct __align__(16) SmemCtl {
  uint64_t full[MAX_STAGES];
  uint64_t empty[MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t xbar[EPI_WARPS];
  uint64_t drain;           // abort path only: completion of the MMAs issued before the abort
  uint64_t bres_full;       // resident B operand has landed
  uint32_t tmem_base;
  int abort_flag;
};

// Position (tm, tn) of tile t of the work list.  CTAs take consecutive tiles, so the tiles in
// flight at one time are a run of the list; the order decides what that run shares in L2.
//   panel_dir 0: row-major over (tm, tn): the run shares few A row blocks and sweeps all of B.
//   panel_dir 1: the tile grid is cut into panels of `panel` tile columns; inside a panel the
//                order is row-major, so the panel's slice of B stays in L2 while A streams past
//                it once per panel.
//   panel_dir 2: panels of `panel` tile rows, column-major inside: the mirror image.
__device__ __forceinline__ void tile_coords(const GemmParams& p, int t, int& tm, int& tn) {
  if (p.panel_dir == 1) {
    const int per = p.tiles_m * p.panel;
    const int pn = t / per, r = t - pn * per;
    const int first = pn * p.panel;
    const int width = (p.tiles_n - first < p.panel) ? p.tiles_n - first : p.panel;
    tm = r / width;
    tn = first + (r - tm * width);
  } else if (p.panel_dir == 2) {
    const int per = p.tiles_n * p.panel;
    const int pm = t / per, r = t - pm * per;
    const int first = pm * p.panel;
    const int height = (p.tiles_m - first < p.panel) ? p.tiles_m - first : p.panel;
    tn = r / height;
    tm = first + (r - tn * height);
  } else {
    tm = t / p.tiles_n;
    tn = t - tm * p.tiles_n;
  }
}

// Contraction block kb of a convolution (modes 1, 2) -> filter tap t and 64-channel chunk cc.  Plain
// order: chunks inside taps.  Column-sharing order: the taps of one filter column are the k-blocks
// of one stage, so blocks run (column, chunk, tap of the column).
__device__ __forceinline__ void conv_block(const GemmParams& p, int kb, int& t, int& cc) {
  if (p.colshare) {
    const int per_col = p.colshare * p.cv.cchunks;
    const int col = kb / per_col, r = kb - col * per_col;
    cc = r / p.colshare;
    t = col * p.colshare + (r - cc * p.colshare);
  } else {
    t = kb / p.cv.cchunks;
    cc = kb - t * p.cv.cchunks;
  }
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// 16-byte piece `piece` (0..3) of row `row` (0..31) inside a 64-byte-swizzled staging block.
__device__ __forceinline__ uint8_t* stg64_addr(uint8_t* base, int row, int piece) {
  return base + row * 64 + ((piece ^ ((row >> 1) & 3)) << 4);
}

template <int A_MN, int B_MN, int EPI, int CTA2>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmX,
            const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmA2,
            const __grid_constant__ CUtensorMap tmA3, const GemmParams p) {
  constexpr bool FWD = (EPI == EPI_FWD || EPI == EPI_FWD_I8);   // forward epilogue (scale, bias)
  constexpr bool I8 = (EPI == EPI_FWD_I8);                       // ... on 8-bit integer operands
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle atoms of TMA and UMMA
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = p.a_region_bytes + p.b_region_bytes;
  uint8_t* bres_reg = smem + p.stages * stage_bytes;         // [nkb][b_stage_bytes] resident B operand (bres)
  uint8_t* out_stg = bres_reg + (p.bres ? p.nkb * p.b_stage_bytes : 0);   // [8 warps][out_bufs][HB_BYTES]
  uint8_t* x_stg = out_stg + (EPI == EPI_PART ? 0 : EPI_WARPS * p.out_bufs * HB_BYTES);   // [8 warps][HB_BYTES] (EPI_DX)
  SmemCtl* ctl = reinterpret_cast<SmemCtl*>(x_stg + (EPI == EPI_DX ? EPI_WARPS * HB_BYTES : 0));
  float* s_scale = reinterpret_cast<float*>(ctl + 1);        // [8 warps][128 scales, 128 biases, 128 zero-point terms] (EPI_FWD), warp-private

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_mn = p.tiles_m * p.tiles_n;
  const int total_items = tiles_mn * p.splits;
  // CTA pair bookkeeping: `rank` inside the pair, `unit` = index of this CTA / pair in the grid
  const int rank = CTA2 ? static_cast<int>(cluster_ctarank()) : 0;
  const int unit = CTA2 ? (blockIdx.x >> 1) : blockIdx.x;
  const int num_units = CTA2 ? (gridDim.x >> 1) : gridDim.x;
  const int TILE_M = CTA2 ? 2 * BM : BM;
  const int bn_cta = CTA2 ? (p.BN >> 1) : p.BN;     // B columns staged by this CTA

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], (CTA2 ? 2 : 1) * EPI_WARPS);
    }
    for (int w = 0; w < EPI_WARPS; ++w) mbar_init(&ctl->xbar[w], 1);
    mbar_init(&ctl->drain, 1);
    mbar_init(&ctl->bres_full, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    if (EPI != EPI_PART) prefetch_tmap(&tmOut);
    if (EPI == EPI_DX) prefetch_tmap(&tmX);
    if (p.cv.mode != 0) {
      prefetch_tmap(&tmA1);
      prefetch_tmap(&tmA2);
      prefetch_tmap(&tmA3);
    }
  }
  if (warp == 1) {
    if (CTA2) {
      tmem_alloc_pair(&ctl->tmem_base, TMEM_COLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(&ctl->tmem_base, TMEM_COLS);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CTA2) cluster_sync();     // the peer's barriers are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  // barriers, TMEM and descriptor prefetches are in place; everything below reads global memory
  // The launch before this one is complete (its writes visible) before this one lets the next
  // launch start.  A launch that reads nothing of its direct predecessor (defer_wait: the
  // weight-gradient GEMM behind the grad-input GEMM, both fed by the prepare launch that the
  // grad-input GEMM has already waited for) starts at once on whatever SMs are free and only
  // holds its exit until the predecessor is done, so that launches behind it still see both.
  if (!p.defer_wait) pdl_wait();
  pdl_trigger();
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    // Lane 0 owns the barrier protocol; the copies of a stage are issued by several lanes at
    // once (a single thread spends ~0.06 us per bulk tensor copy, which bounds narrow tiles).
    // Lanes 0..5 take the merged MN-major boxes (A chunks 0-1, B chunks 0-3); lanes 8.. take
    // the per-k-block copies, two lanes per k-block (A operand, B operand).
    {
      int it = 0, ring_s = 0;
      uint32_t ring_ph = 0;
      bool live = true;
      const uint64_t pol_a = l2_policy(p.hint_a), pol_b = l2_policy(p.hint_b);
      if (p.bres && unit < total_items) {
        // resident B operand: every (tap, chunk) block once, all on one barrier
        const int bch = (((static_cast<int>(p.Nc) + 15) & ~15) + 63) >> 6;
        const uint32_t tx_b1 = B_MN ? bch * CHUNK_BYTES : bn_cta * BK * 2;
        if (lane == 0) mbar_arrive_expect_tx(&ctl->bres_full, tx_b1 * p.nkb);
        __syncwarp();
        for (int kb = lane; kb < p.nkb; kb += 32) {
          int t, cc;
          conv_block(p, kb, t, cc);
          const int rs = p.cv.tap_rs[t];
          uint8_t* sb = bres_reg + kb * p.b_stage_bytes;
          if (B_MN) {
            for (int c = 0; c < bch; ++c)
              tma_load_2d(sb + c * CHUNK_BYTES, &tmB, &ctl->bres_full, rs * p.cv.wcols + 64 * c, cc * 64);
          } else {
            tma_load_2d(sb, &tmB, &ctl->bres_full, rs * p.cv.wcols + cc * 64, 0);
          }
        }
      }
      for (int w = unit; w < total_items && live; w += num_units) {
        const int split = w / tiles_mn, t = w - split * tiles_mn;
        int tm, tn;
        tile_coords(p, t, tm, tn);
        const int m0 = tm * TILE_M + rank * BM;
        const int n0 = tn * p.BN + rank * bn_cta;     // first B column staged by this CTA
        int n_eff = static_cast<int>(p.Nc - n0);
        if (n_eff > bn_cta) n_eff = bn_cta;
        n_eff = (n_eff + 15) & ~15;
        const int b_chunks = (n_eff + 63) >> 6;
        // bytes credited to the (leader's) full barrier per stage: both CTAs' copies in pair mode
        // (a merged MN-major box always brings all kps k-blocks of its chunk, used or not)
        const uint32_t tx_a = A_STAGE_BYTES, tx_b = p.bres ? 0u : (B_MN ? b_chunks * CHUNK_BYTES : bn_cta * BK * 2);
        const bool a_mrg = A_MN && p.merged, b_mrg = B_MN && p.merged;
        const int kb_begin = static_cast<int>(static_cast<int64_t>(split) * p.nkb / p.splits);
        const int kb_end = static_cast<int>(static_cast<int64_t>(split + 1) * p.nkb / p.splits);
        // One barrier round trip costs ~0.3 us whatever it carries, so a stage holds several
        // k-blocks: all of them land on the same full barrier and are released by one commit.
        // convolution (modes 1, 2): filter tap and channel chunk of this lane's k-block, kept by
        // increments from stage to stage (an integer division per copy sat on the issue path)
        int ct = 0, ccc = 0, tw0 = 0, th0 = 0, tb0 = 0;     // ... and the origin of the tile's pixel box
        if ((p.cv.mode == 1 || p.cv.mode == 2) && lane >= 8) {
          conv_block(p, kb_begin + ((lane - 8) >> 1), ct, ccc);
          const int bw = tm % p.cv.tiles_w, bh = (tm / p.cv.tiles_w) % p.cv.tiles_h;
          const int bb = tm / (p.cv.tiles_w * p.cv.tiles_h);
          tw0 = bw * p.cv.tw; th0 = bh * p.cv.th; tb0 = bb * p.cv.tb;
        }
        // grad-weight: contraction block -> box of 64 output pixels, and the (tap, first channel) of
        // the two 64-row halves of this tile
        int kbw = 0, kbh = 0, kbb = 0, at[2] = {0, 0}, ac[2] = {0, 0};
        if (p.cv.mode == 3 && lane >= 8) {
          const int kb = kb_begin + ((lane - 8) >> 1);
          kbw = kb % p.cv.tiles_w; kbh = (kb / p.cv.tiles_w) % p.cv.tiles_h;
          kbb = kb / (p.cv.tiles_w * p.cv.tiles_h);
          const int cpad = p.cv.cchunks * 64;       // tile rows per tap (channels padded to 64)
          for (int j = 0; j < 2; ++j) {
            const int k = m0 + 64 * j;
            at[j] = k / cpad; ac[j] = k - at[j] * cpad;
            if (at[j] >= p.cv.ntaps) { at[j] = 0; ac[j] = p.cv.C; }     // past the last tap: all zeros
          }
        }
        for (int kb0 = kb_begin; kb0 < kb_end; kb0 += p.kps, ++it, ring_s = (ring_s + 1 == p.stages) ? 0 : ring_s + 1,
                 ring_ph ^= (ring_s == 0) ? 1u : 0u) {
          const int nsub = (kb_end - kb0 < p.kps) ? kb_end - kb0 : p.kps;
          const int s = ring_s;               // it % stages and (it / stages) & 1, kept by increments
          const uint32_t ph = ring_ph;
          int ok_stage = 1;
          if (lane == 0) {
            if (*abort_flag || !mbar_wait(&ctl->empty[s], ph ^ 1)) {
              record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
              *abort_flag = 1;
              ok_stage = 0;
            } else if (rank == 0) {
              // the leader's barrier collects the bytes of both CTAs of a pair; only the leader arrives on it
              mbar_arrive_expect_tx(&ctl->full[s], (CTA2 ? 2u : 1u) * ((p.colshare ? static_cast<uint32_t>(p.a_tx)
                                                                                   : tx_a * (a_mrg ? p.kps : nsub)) +
                                                                      tx_b * (b_mrg ? p.kps : nsub)));
            }
          }
          ok_stage = __shfl_sync(0xffffffffu, ok_stage, 0);
          if (!ok_stage) {
            live = false;
            break;
          }
          uint8_t* a_reg = smem + s * stage_bytes;               // [kps k-blocks of A][kps k-blocks of B]
          uint8_t* b_reg = a_reg + p.a_region_bytes;
          const uint32_t fb = CTA2 ? mapa_u32(smem_u32(&ctl->full[s]), 0) : 0u;
          if (lane < 6) {
            // one box of kps * 64 contraction rows per 64-wide chunk: chunk c sits at c * kps * 8 KiB
            const int chunk_stride = p.kps * CHUNK_BYTES;
            if (a_mrg && lane < 2) {
              const int c = lane;
              if (CTA2) tma_load_2d_pair_hint(a_reg + c * chunk_stride, &tmA, fb, m0 + 64 * c, kb0 * BK, pol_a);
              else tma_load_2d_hint(a_reg + c * chunk_stride, &tmA, &ctl->full[s], m0 + 64 * c, kb0 * BK, pol_a);
            }
            if (b_mrg && lane >= 2 && lane - 2 < b_chunks) {
              const int c = lane - 2;
              if (CTA2) tma_load_2d_pair_hint(b_reg + c * chunk_stride, &tmB, fb, n0 + 64 * c, kb0 * BK, pol_b);
              else tma_load_2d_hint(b_reg + c * chunk_stride, &tmB, &ctl->full[s], n0 + 64 * c, kb0 * BK, pol_b);
            }
          }
          const int u = (lane - 8) >> 1;
          const bool do_a = lane >= 8 && u < nsub && !(lane & 1) && !a_mrg;
          const bool do_b = lane >= 8 && u < nsub && (lane & 1) && !b_mrg;
          if (do_a || do_b) {
            const int kb = kb0 + u;
            uint8_t* sa = a_reg + u * A_STAGE_BYTES;
            uint8_t* sb = b_reg + u * p.b_stage_bytes;
            if (CTA2) {
              if (do_a) {
                if (A_MN) {
                  tma_load_2d_pair_hint(sa, &tmA, fb, m0, kb * BK, pol_a);
                  tma_load_2d_pair_hint(sa + CHUNK_BYTES, &tmA, fb, m0 + 64, kb * BK, pol_a);
                } else {
                  tma_load_2d_pair_hint(sa, &tmA, fb, kb * p.bk, m0, pol_a);
                }
              } else {
                if (B_MN) {
                  for (int c = 0; c < b_chunks; ++c)
                    tma_load_2d_pair_hint(sb + c * CHUNK_BYTES, &tmB, fb, n0 + 64 * c, kb * BK, pol_b);
                } else {
                  tma_load_2d_pair_hint(sb, &tmB, fb, kb * p.bk, n0, pol_b);
                }
              }
            } else if (p.cv.mode == 0) {
              if (do_a) {
                if (A_MN) {
                  tma_load_2d_hint(sa, &tmA, &ctl->full[s], m0, kb * BK, pol_a);
                  tma_load_2d_hint(sa + CHUNK_BYTES, &tmA, &ctl->full[s], m0 + 64, kb * BK, pol_a);
                } else {
                  tma_load_2d_hint(sa, &tmA, &ctl->full[s], kb * p.bk, m0, pol_a);
                }
              } else {
                if (B_MN) {
                  for (int c = 0; c < b_chunks; ++c)
                    tma_load_2d_hint(sb + c * CHUNK_BYTES, &tmB, &ctl->full[s], n0 + 64 * c, kb * BK, pol_b);
                } else {
                  tma_load_2d_hint(sb, &tmB, &ctl->full[s], kb * p.bk, n0, pol_b);
                }
              }
            } else if (p.cv.mode == 3) {
              // grad-weight: contraction block kb = one box of 64 output pixels; tile rows = (tap, channel)
              const int w0 = kbw * p.cv.tw, h0 = kbh * p.cv.th, b0 = kbb * p.cv.tb;
              if (do_a) {
                for (int j = 0; j < 2; ++j) {
                  const int t = at[j], c = ac[j];
                  const int mi = p.cv.tap_map[t];
                  const CUtensorMap* ma = mi == 0 ? &tmA : (mi == 1 ? &tmA1 : (mi == 2 ? &tmA2 : &tmA3));
                  tma_load_4d(sa + j * CHUNK_BYTES, ma, &ctl->full[s], c, w0 + p.cv.tap_dw[t], h0 + p.cv.tap_dh[t], b0);
                }
              } else {
                for (int c = 0; c < b_chunks; ++c)
                  tma_load_4d(sb + c * CHUNK_BYTES, &tmB, &ctl->full[s], n0 + 64 * c, w0, h0, b0);
              }
            } else {
              // forward / grad-input: tile rows = one box of 128 pixels; contraction block kb = (tap, 64 channels)
              const int w0 = tw0, h0 = th0, b0 = tb0;
              const int t = ct, cc = ccc;
              const int rs = p.cv.tap_rs[t];
              if (do_a) {
                if (p.colshare) {
                  // the first tap of the filter column (smallest row shift) brings the box of all of them
                  if (u == 0) {
                    const int mi = p.cv.tap_map[t];
                    const CUtensorMap* ma = mi == 0 ? &tmA : (mi == 1 ? &tmA1 : (mi == 2 ? &tmA2 : &tmA3));
                    tma_load_4d(a_reg, ma, &ctl->full[s], cc * 64, w0 + p.cv.tap_dw[t], h0 + p.cv.tap_dh[t], b0);
                  }
                } else {
                  const int mi = p.cv.tap_map[t];
                  const CUtensorMap* ma = mi == 0 ? &tmA : (mi == 1 ? &tmA1 : (mi == 2 ? &tmA2 : &tmA3));
                  tma_load_4d(sa, ma, &ctl->full[s], cc * 64, w0 + p.cv.tap_dw[t], h0 + p.cv.tap_dh[t], b0);
                }
              } else if (p.bres) {
                // B operand already resident
              } else if (B_MN) {     // W^ viewed as [N rows, R*S*Cin columns]: rows = contraction
                for (int c = 0; c < b_chunks; ++c)
                  tma_load_2d(sb + c * CHUNK_BYTES, &tmB, &ctl->full[s], rs * p.cv.wcols + n0 + 64 * c, cc * 64);
              } else {               // weight codes [N, R*S*Cin]: columns past this tap's channels meet zeros of A
                tma_load_2d(sb, &tmB, &ctl->full[s], rs * p.cv.wcols + cc * 64, n0);
              }
            }
          }
          if (p.cv.mode == 3) {
            kbw += p.kps;
            while (kbw >= p.cv.tiles_w) {
              kbw -= p.cv.tiles_w;
              if (++kbh == p.cv.tiles_h) { kbh = 0; ++kbb; }
            }
          } else if (p.colshare) {
            if (++ccc == p.cv.cchunks) { ccc = 0; ct += p.colshare; }
          } else {
            ccc += p.kps;
            while (ccc >= p.cv.cchunks && p.cv.cchunks > 0) { ccc -= p.cv.cchunks; ++ct; }
          }
          __syncwarp();
        }
      }
      // Make sure none of this CTA's bulk copies is still in flight when it exits (only
      // relevant after an abort: otherwise the MMA warp has consumed every stage).
      const int issued = it;
      if (lane == 0 && rank == 0) {
        for (int j = (issued > p.stages ? issued - p.stages : 0); j < issued; ++j)
          mbar_wait(&ctl->full[j % p.stages], (j / p.stages) & 1, 20000000ull);
        if (p.bres && unit < total_items) mbar_wait(&ctl->bres_full, 0, 20000000ull);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0 && rank == 0) {
      int it = 0, acc_it = 0, ring_s = 0;
      uint32_t ring_ph = 0;
      bool ok = true;
      // This one thread is the critical path of tiles with few or narrow MMAs, so nothing it does per
      // tile or per instruction is more than it must be: the tile's position is only computed when
      // tiles differ in width (a ragged last tile column), the k-range only for split contractions
      // (both need integer divisions), and the operand descriptors of a k-block are built once and
      // advanced by adding to their address field.
      // (one tile column: every tile has the same width, ragged or not)
      const bool ragged_n = p.tiles_n > 1 && (p.Nc % p.BN) != 0;
      const int n_first = static_cast<int>(((p.Nc < p.BN ? p.Nc : p.BN) + 15) & ~static_cast<int64_t>(15));
      const uint32_t idesc_full = I8 ? instr_desc_i8(TILE_M, n_first, p.a_signed, 1) : instr_desc_bf16(TILE_M, n_first, A_MN, B_MN);
      const bool a_mrg = A_MN && p.merged, b_mrg = B_MN && p.merged;
      const uint32_t a_lbo = a_mrg ? p.kps * CHUNK_BYTES : CHUNK_BYTES;
      const uint32_t b_lbo = b_mrg ? p.kps * CHUNK_BYTES : CHUNK_BYTES;
      const uint32_t a_step = a_mrg ? CHUNK_BYTES : p.a_sub_off;
      const uint32_t b_step = b_mrg ? CHUNK_BYTES : p.b_stage_bytes;
      const uint32_t bres_base = smem_u32(bres_reg);
      const uint32_t ring_base = smem_u32(smem);
      for (int w = unit; w < total_items && ok; w += num_units, ++acc_it) {
        uint32_t idesc = idesc_full;
        int kb_begin = 0, kb_end = p.nkb;
        if (ragged_n || p.splits > 1) {
          const int split = w / tiles_mn, t = w - split * tiles_mn;
          int tm, tn;
          tile_coords(p, t, tm, tn);
          const int n0 = tn * p.BN;
          int n_eff = static_cast<int>(p.Nc - n0);
          if (n_eff > p.BN) n_eff = p.BN;
          n_eff = (n_eff + 15) & ~15;
          idesc = I8 ? instr_desc_i8(TILE_M, n_eff, p.a_signed, 1) : instr_desc_bf16(TILE_M, n_eff, A_MN, B_MN);
          if (p.splits > 1) {
            kb_begin = static_cast<int>(static_cast<int64_t>(split) * p.nkb / p.splits);
            kb_end = static_cast<int>(static_cast<int64_t>(split + 1) * p.nkb / p.splits);
          }
        }
        const int buf = acc_it & 1;
        // wait until the epilogue has drained this accumulator (two tiles ago)
        if (*abort_flag || !mbar_wait(&ctl->acc_empty[buf], ((acc_it >> 1) & 1) ^ 1)) {
          record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
          *abort_flag = 1;
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * ACC_STRIDE;
        if (p.bres && acc_it == 0) {
          if (*abort_flag || !mbar_wait(&ctl->bres_full, 0)) {
            record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
            *abort_flag = 1;
            ok = false;
            break;
          }
        }
        for (int kb0 = kb_begin; kb0 < kb_end; kb0 += p.kps, ++it, ring_s = (ring_s + 1 == p.stages) ? 0 : ring_s + 1,
                 ring_ph ^= (ring_s == 0) ? 1u : 0u) {
          const int nsub = (kb_end - kb0 < p.kps) ? kb_end - kb0 : p.kps;
          const int s = ring_s;               // it % stages and (it / stages) & 1, kept by increments
          const uint32_t ph = ring_ph;
          if (*abort_flag || !mbar_wait(&ctl->full[s], ph)) {
            record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
            *abort_flag = 1;
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_base = ring_base + s * stage_bytes;
          const uint32_t b_base = p.bres ? bres_base + kb0 * p.b_stage_bytes : a_base + p.a_region_bytes;
         for (int u = 0; u < nsub; ++u) {
          const int kb = kb0 + u;
          // k-block u of the stage: merged MN-major operands keep their chunks kps * 8 KiB apart
          const uint32_t a_addr = a_base + u * a_step;
          const uint32_t b_addr = b_base + u * b_step;
          // K-major: 16 contraction elements = 32 bytes inside the swizzled 128-byte row.
          // MN-major: 16 contraction elements = 16 rows of 128 bytes = two 8-row groups.
          // The address field counts 16-byte units and cannot carry out of its 14 bits (shared
          // memory ends below 256 KiB), so a k-step is an addition to the whole descriptor.
          const uint64_t adesc0 = A_MN ? smem_desc_sw128(a_addr, a_lbo, 1024) : smem_desc_sw128(a_addr, 16, 1024);
          const uint64_t bdesc0 = B_MN ? smem_desc_sw128(b_addr, b_lbo, 1024) : smem_desc_sw128(b_addr, 16, 1024);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = adesc0 + static_cast<uint64_t>(k * (A_MN ? 2048 / 16 : 32 / 16));
            const uint64_t bdesc = bdesc0 + static_cast<uint64_t>(k * (B_MN ? 2048 / 16 : 32 / 16));
            const uint32_t accum = (kb > kb_begin || k > 0) ? 1u : 0u;
            if (I8) {
              if (CTA2) umma_i8_pair(d_tmem, adesc, bdesc, idesc, accum); else umma_i8(d_tmem, adesc, bdesc, idesc, accum);
            } else {
              if (CTA2) umma_bf16_pair(d_tmem, adesc, bdesc, idesc, accum); else umma_bf16(d_tmem, adesc, bdesc, idesc, accum);
            }
          }
         }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (CTA2) umma_commit_pair(&ctl->empty[s], 3); else umma_commit(&ctl->empty[s]);
        }
        if (ok) {
          if (CTA2) umma_commit_pair(&ctl->acc_full[buf], 3); else umma_commit(&ctl->acc_full[buf]);
        }
      }
      if (!ok) {
        // MMAs issued before the abort may still be reading the ring and writing TMEM: nothing
        // of this CTA is torn down before they have completed (own barrier only, bounded)
        if (CTA2) umma_commit_pair(&ctl->drain, 1); else umma_commit(&ctl->drain);
        mbar_wait(&ctl->drain, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------- epilogue (warps 2..9)
    // Warp e = warp - 2 reads TMEM lane quarter q = warp % 4 (the quarter the hardware lets
    // it read) and owns one half of the tile's column blocks.  A block is 64 bytes of output
    // columns (32 bf16 / 16 fp32): small enough that two staging buffers per warp fit, so the
    // TMA store of one block drains while the next one is computed.
    const int e = warp - 2;
    const int q = warp & 3;
    const int half = e >> 2;
    const int bc = p.blk_cols;
    uint8_t* my_out = out_stg + e * p.out_bufs * HB_BYTES;
    uint8_t* my_x = x_stg + e * HB_BYTES;
    float* my_sc = s_scale + e * 384;          // [128] scales, [128] biases, [128] Zr * wsum (as int) of this warp's columns
    int* my_zw = reinterpret_cast<int*>(my_sc + 256);
    ActQ xq = {};
    if (EPI != EPI_PART) xq = make_actq(p.s_x, p.z_x, p.x_bits, p.x_sym, nullptr);
    const int zr_i = static_cast<int>(xq.zr);
    const float t_lo = xq.lo - xq.zr, t_hi = xq.hi - xq.zr;     // d/ds of a clipped element
    const float q_half = 0.5f * (xq.hi - xq.lo), z_mid = xq.zr - 0.5f * (xq.hi + xq.lo);

    struct Geo {
      int t, split, n0, n_eff, row0, jb0, jb1, pw0, ph0, pb0;
      bool rows_live;
    };
    auto geo_of = [&](int w) {
      Geo g;
      g.split = w / tiles_mn;
      g.t = w - g.split * tiles_mn;
      int tm, tn;
      tile_coords(p, g.t, tm, tn);
      const int m0 = tm * TILE_M + rank * BM;
      g.n0 = tn * p.BN;
      int n_eff = static_cast<int>(p.Nc - g.n0);
      if (n_eff > p.BN) n_eff = p.BN;
      g.n_eff = (n_eff + 15) & ~15;
      const int bw_cols = (EPI == EPI_PART) ? 32 : bc;
      const int nblk = (g.n_eff + bw_cols - 1) / bw_cols;
      const int nb0 = (nblk + 1) >> 1;
      g.jb0 = half ? nb0 : 0;
      g.jb1 = half ? nblk : nb0;
      g.row0 = m0 + q * 32;
      g.pw0 = g.ph0 = g.pb0 = 0;
      g.rows_live = g.row0 < p.Mr;
      if (EPI != EPI_PART && p.cv.mode != 0) {
        // convolution: this warp's 32 rows are a sub-box of the tile's pixel box
        const int tmi = tm;
        const int bw = tmi % p.cv.tiles_w, bh = (tmi / p.cv.tiles_w) % p.cv.tiles_h;
        const int bb = tmi / (p.cv.tiles_w * p.cv.tiles_h);
        const int pix = q * 32;
        g.pw0 = bw * p.cv.tw;
        g.ph0 = bh * p.cv.th + (pix / p.cv.tw) % p.cv.th;
        g.pb0 = bb * p.cv.tb + pix / (p.cv.tw * p.cv.th);
        g.rows_live = g.ph0 < p.cv.dimH && g.pb0 < p.cv.dimB;
      }
      return g;
    };
    int x_issued = 0;                        // X blocks requested so far (lane 0 only)
    auto fetch_x = [&](const Geo& g, int jb) {     // lane 0: one 32-row x 64-byte block of X
      uint64_t* xb = &ctl->xbar[e];
      ++x_issued;
      mbar_arrive_expect_tx(xb, HB_BYTES);
      if (p.cv.mode != 0) tma_load_4d(my_x, &tmX, xb, g.n0 + jb * bc, g.pw0, g.ph0, g.pb0);
      else tma_load_2d(my_x, &tmX, xb, g.n0 + jb * bc, g.row0);
    };

    int acc_it = 0;
    int x_it = 0;                            // X blocks consumed so far by this warp (EPI_DX)
    int st_it = 0;                           // output blocks staged so far by this warp
    bool ok = true;
    Geo g = {};
    if (unit < total_items) {
      g = geo_of(unit);
      if (EPI == EPI_DX && lane == 0 && g.jb0 < g.jb1) fetch_x(g, g.jb0);
      if (FWD) {
        for (int j = lane; j < 128; j += 32) {
          const int64_t c = static_cast<int64_t>(g.n0) + g.jb0 * bc + j;
          my_sc[j] = (c < p.Nc) ? p.col_scale[c] * xq.s : 0.f;
          my_sc[128 + j] = (c < p.Nc && p.col_bias) ? p.col_bias[c] : 0.f;
          if (I8) my_zw[j] = (c < p.Nc) ? zr_i * p.wsum[c] : 0;
        }
        __syncwarp();
      }
    }
    for (int w = unit; w < total_items && ok; w += num_units, ++acc_it) {
      const bool has_next = w + num_units < total_items;
      const Geo gn = has_next ? geo_of(w + num_units) : g;
      const int buf = acc_it & 1;
      // next tile's column scales and biases: loaded now, parked in registers behind this tile's work
      float nsc[4] = {0.f, 0.f, 0.f, 0.f}, nbi[4] = {0.f, 0.f, 0.f, 0.f};
      int nzw[4] = {0, 0, 0, 0};
      // (a tile list with one tile column keeps the same scales from tile to tile: nothing to load)
      const bool new_cols = has_next && (gn.n0 != g.n0 || gn.jb0 != g.jb0);
      if (FWD && new_cols) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int64_t c = static_cast<int64_t>(gn.n0) + gn.jb0 * bc + lane + 32 * i;
          if (c < p.Nc) {
            nsc[i] = p.col_scale[c] * xq.s;
            if (p.col_bias) nbi[i] = p.col_bias[c];
            if (I8) nzw[i] = zr_i * p.wsum[c];
          }
        }
      }
      bool got = *abort_flag ? false : mbar_wait(&ctl->acc_full[buf], (acc_it >> 1) & 1);
      got = __all_sync(0xffffffffu, got);
      if (!got) {
        record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
        *abort_flag = 1;
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + buf * ACC_STRIDE + (static_cast<uint32_t>(q * 32) << 16);
      float acc_s = 0.f, acc_c = 0.f;

      if (EPI == EPI_PART) {
        int64_t row = static_cast<int64_t>(g.row0) + lane;
        if (p.cv.mode == 3) {
          // tile row (tap, channel padded to 64) -> row of the weight matrix; padding rows are skipped
          const int cpad = p.cv.cchunks * 64;
          const int t = static_cast<int>(row) / cpad, c = static_cast<int>(row) - t * cpad;
          row = (t < p.cv.ntaps && c < p.cv.C) ? static_cast<int64_t>(p.cv.tap_rs[t]) * p.cv.C + c : p.Mr;
        }
        for (int jb = g.jb0; jb < g.jb1; ++jb) {
          const int c0 = jb * 32;
          uint32_t r[32];
          const int ncols = (g.n_eff - c0 >= 32) ? 32 : 16;
          if (ncols == 32) tmem_ld_32x32(t_row + c0, r); else tmem_ld_32x16(t_row + c0, r);
          tmem_wait_ld();
          if (row < p.Mr) {
            float* outp = p.out + g.split * p.split_stride + row;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int64_t col = static_cast<int64_t>(g.n0) + c0 + j;
              if (j < ncols && col < p.part_cols) outp[col * p.ldo] = __uint_as_float(r[j]);
            }
          }
        }
      } else {
        for (int jb = g.jb0; jb < g.jb1 && ok; ++jb) {
          const int c0 = jb * bc;
          const int left = g.n_eff - c0;
          const int ncols = (left >= 32 && bc == 32) ? 32 : 16;
          uint4 xr[4];      // this thread's row of the X block: 4 pieces of 16 bytes
          if (EPI == EPI_DX) {
            bool gx = mbar_wait(&ctl->xbar[e], x_it & 1);
            gx = __all_sync(0xffffffffu, gx);
            if (!gx) {
              record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
              *abort_flag = 1;
              ok = false;
              break;
            }
            ++x_it;
#pragma unroll
            for (int i = 0; i < 4; ++i) xr[i] = *reinterpret_cast<const uint4*>(stg64_addr(my_x, lane, i));
            // The next bulk copy overwrites this buffer through the async proxy.  Plain barriers do
            // not order generic-proxy reads against it (the loads may legally be delayed up to
            // their first use, far behind the copy's issue): the proxy fence does.
            fence_proxy_async();
            __syncwarp();
            // the block now lives in registers: fetch the next one (of this or the next tile) behind the math
            if (lane == 0) {
              if (jb + 1 < g.jb1) fetch_x(g, jb + 1);
              else if (has_next && gn.jb0 < gn.jb1) fetch_x(gn, gn.jb0);
            }
          }
          uint32_t r[32];
          if (ncols == 32) tmem_ld_32x32(t_row + c0, r); else tmem_ld_32x16(t_row + c0, r);
          float4 sc4[8], bi4[8];     // this block's column scales (s_x folded in) and biases
          if (FWD) {
            const float4* ps = reinterpret_cast<const float4*>(my_sc + (jb - g.jb0) * bc);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              if (i * 4 < bc) {
                sc4[i] = ps[i];
                bi4[i] = ps[32 + i];
              }
            }
          }
          // the TMA store that last used this staging buffer must have finished reading it
          uint8_t* ob = my_out + (p.out_bufs == 2 ? (st_it & 1) * HB_BYTES : 0);
          if (lane == 0) {
            if (p.out_bufs == 2) tma_store_wait_read1(); else tma_store_wait_read0();
          }
          ++st_it;
          tmem_wait_ld();
          __syncwarp();
#pragma unroll
          for (int gi = 0; gi < 4; ++gi) {
            if (gi * 8 < ncols) {
              float v[8];
              if (FWD) {
                const float sv[8] = {sc4[2 * gi].x, sc4[2 * gi].y, sc4[2 * gi].z, sc4[2 * gi].w,
                                     sc4[2 * gi + 1].x, sc4[2 * gi + 1].y, sc4[2 * gi + 1].z, sc4[2 * gi + 1].w};
                const float bv[8] = {bi4[2 * gi].x, bi4[2 * gi].y, bi4[2 * gi].z, bi4[2 * gi].w,
                                     bi4[2 * gi + 1].x, bi4[2 * gi + 1].y, bi4[2 * gi + 1].z, bi4[2 * gi + 1].w};
                if (I8) {
                  // integer accumulators: sum_k q_x q_w - Zr sum_k q_w = sum_k (q_x - Zr) q_w, exact in int32
                  const int4* pz = reinterpret_cast<const int4*>(my_zw + (jb - g.jb0) * bc) + 2 * gi;
                  const int4 z0 = pz[0], z1 = pz[1];       // Zr * (row sum of the weight codes) of these columns
                  const int zv[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
#pragma unroll
                  for (int j = 0; j < 8; ++j)
                    v[j] = fmaf(static_cast<float>(static_cast<int>(r[gi * 8 + j]) - zv[j]), sv[j], bv[j]);
                } else {
#pragma unroll
                  for (int j = 0; j < 8; ++j) v[j] = fmaf(__uint_as_float(r[gi * 8 + j]), sv[j], bv[j]);
                }
              } else {
                float x[8];
                if (bc == 32) {      // bf16 activations: 8 values in one 16-byte piece
                  const uint4 u = xr[gi];
                  const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    x[2 * i] = __uint_as_float(wv[i] << 16);
                    x[2 * i + 1] = __uint_as_float(wv[i] & 0xffff0000u);
                  }
                } else {             // fp32 activations: two 16-byte pieces
                  const uint4 a = xr[(2 * gi) & 3], b = xr[(2 * gi + 1) & 3];
                  x[0] = __uint_as_float(a.x); x[1] = __uint_as_float(a.y);
                  x[2] = __uint_as_float(a.z); x[3] = __uint_as_float(a.w);
                  x[4] = __uint_as_float(b.x); x[5] = __uint_as_float(b.y);
                  x[6] = __uint_as_float(b.z); x[7] = __uint_as_float(b.w);
                }
                // Eq. 1 with the straight-through estimator, the arithmetic of quant_act().  An
                // element is clipped iff |rne(x/s) + Z - mid| > half (all operands are multiples
                // of 0.5 below 2^23: exact).  Groups in which no lane of the warp has a clipped
                // element skip the selects and the zero-point sum.
                float rq[8], dq[8];
                bool any_clip = false;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  rq[j] = rne_small(__fmul_rn(x[j], xq.rinv));
                  dq[j] = rq[j] + z_mid;
                  any_clip = any_clip || fabsf(dq[j]) > q_half;
                }
                if (!__any_sync(0xffffffffu, any_clip)) {
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const float gx = __uint_as_float(r[gi * 8 + j]);
                    const float resid = fmaf(-x[j], xq.rinv_lo, fmaf(-x[j], xq.rinv, rq[j]));
                    v[j] = gx;
                    acc_s = fmaf(gx, resid, acc_s);
                  }
                } else {
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const float gx = __uint_as_float(r[gi * 8 + j]);
                    const bool clipped = fabsf(dq[j]) > q_half;
                    const float resid = fmaf(-x[j], xq.rinv_lo, fmaf(-x[j], xq.rinv, rq[j]));
                    const float tq = clipped ? (dq[j] < 0.f ? t_lo : t_hi) : resid;
                    v[j] = clipped ? 0.f : gx;
                    acc_s = fmaf(gx, tq, acc_s);
                    acc_c += clipped ? gx : 0.f;
                  }
                }
              }
              if (bc == 32) {
                uint4 o;
                o.x = pack2(v[0], v[1]); o.y = pack2(v[2], v[3]);
                o.z = pack2(v[4], v[5]); o.w = pack2(v[6], v[7]);
                *reinterpret_cast<uint4*>(stg64_addr(ob, lane, gi)) = o;
              } else {
                *reinterpret_cast<float4*>(stg64_addr(ob, lane, 2 * gi)) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4*>(stg64_addr(ob, lane, 2 * gi + 1)) = make_float4(v[4], v[5], v[6], v[7]);
              }
            }
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (g.rows_live && g.n0 + c0 < p.Nc) {     // stores are clipped at the tensor's edges
              if (p.cv.mode != 0) tma_store_4d(&tmOut, ob, g.n0 + c0, g.pw0, g.ph0, g.pb0);
              else tma_store_2d(&tmOut, ob, g.n0 + c0, g.row0);
            }
            tma_store_commit();     // always: the buffer rotation counts committed groups
          }
        }
      }
      // every TMEM read of this accumulator is complete: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTA2) mbar_arrive_cluster(mapa_u32(smem_u32(&ctl->acc_empty[buf]), 0));   // leader's barrier
        else mbar_arrive(&ctl->acc_empty[buf]);
      }
      if (EPI == EPI_DX && ok) {
        acc_s = warp_sum(acc_s);
        acc_c = warp_sum(acc_c);
        if (lane == 0) {
          float* pp = p.partials + ((static_cast<int64_t>(g.t) * (CTA2 ? 2 : 1) + rank) * EPI_WARPS + e) * 2;
          pp[0] = acc_s;
          pp[1] = -xq.s * acc_c;     // Eq. 1: d(dequantised)/dZ = -s on clipped elements, 0 elsewhere
        }
      }
      if (FWD && new_cols) {
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          my_sc[lane + 32 * i] = nsc[i];
          my_sc[128 + lane + 32 * i] = nbi[i];
          if (I8) my_zw[lane + 32 * i] = nzw[i];
        }
        __syncwarp();
      }
      g = gn;
    }
    // after an abort a requested X block may still be on its way into this warp's buffer
    if (EPI == EPI_DX && !ok && lane == 0 && x_issued > x_it) mbar_wait(&ctl->xbar[e], x_it & 1, 20000000ull);
    if (EPI != EPI_PART && lane == 0) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (CTA2) cluster_sync();     // neither CTA leaves while its peer may still signal its barriers
  if (p.defer_wait && threadIdx.x == 0) pdl_wait();
  if (warp == 1) {
    if (CTA2) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once (a constant of the process, not state).
static EncodeTiledFn tensor_map_encoder() {
  static const EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess || !f ||
        qres != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// 2-D row-major matrix [rows, cols] with pitch ld (elements); box = row_bytes (128 or 64, the
// swizzle span) of columns x box_rows rows.  is_bf16: 0 fp32, 1 bf16, 2 8-bit integer.
static int make_map(CUtensorMap* m, const void* base, int is_bf16, int64_t rows, int64_t cols, int64_t ld,
                    int box_rows, int row_bytes = 128) {
  const int es = (is_bf16 == 2) ? 1 : (is_bf16 ? 2 : 4);
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * es};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(row_bytes / es), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUtensorMapDataType dt = (is_bf16 == 2) ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                 : (is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32);
  const CUresult r = tensor_map_encoder()(m, dt, 2,
                              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? EFQAT_OK : EFQAT_ERR_CUDA;
}

int tensor_map_2d(CUtensorMap* m, const void* base, int kind, int64_t rows, int64_t cols, int64_t ld, int box_rows,
                  int row_bytes) {
  if (!tensor_map_encoder()) return EFQAT_ERR_CUDA;
  return make_map(m, base, kind, rows, cols, ld, box_rows, row_bytes);
}

// 4-D NHWC tensor [B,H,W,C] (pitch C elements per pixel); box = row_bytes (128 or 64) of channels x bw x bh x bb pixels.
// sw / sh / sb: distance in elements between neighbouring pixels along W, H and B (0: dense,
// i.e. pitch, pitch * W, pitch * W * H).  A strided convolution addresses one of its
// stride x stride interleaved pixel sub-grids this way: base moved to the sub-grid's first
// pixel, W and H counted in sub-grid pixels, sw and sh multiplied by the stride.
static int make_map_4d(CUtensorMap* m, const void* base, int is_bf16, int64_t B, int64_t H, int64_t W, int64_t C,
                       int64_t pitch, int bw, int bh, int bb, int row_bytes = 128, int64_t sw = 0, int64_t sh = 0,
                       int64_t sb = 0) {
  const int es = is_bf16 ? 2 : 4;
  if (!sw) sw = pitch;
  if (!sh) sh = pitch * W;
  if (!sb) sb = pitch * W * H;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(H),
                              static_cast<cuuint64_t>(B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(sw) * es, static_cast<cuuint64_t>(sh) * es,
                                 static_cast<cuuint64_t>(sb) * es};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(row_bytes / es), static_cast<cuuint32_t>(bw),
                             static_cast<cuuint32_t>(bh), static_cast<cuuint32_t>(bb)};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = tensor_map_encoder()(m, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? EFQAT_OK : EFQAT_ERR_CUDA;
}

// Pixel box (power-of-two sides, tw * th * tb = target) that wastes the least work on a
// W x H x B pixel space; tw <= 32 so that a quarter of a 128-pixel box is a sub-box.
void conv_pixel_box(int W, int H, int B, int target, int* tw, int* th, int* tb) {
  double best = 1e300;
  *tw = 1; *th = 1; *tb = target;
  for (int a = 1; a <= target && a <= 32; a <<= 1)
    for (int b = 1; a * b <= target; b <<= 1) {
      const int c = target / (a * b);
      const double vol = static_cast<double>(ceil_div(W, a) * a) * static_cast<double>(ceil_div(H, b) * b) *
                         static_cast<double>(ceil_div(B, c) * c);
      // prefer wider boxes at equal volume: longer contiguous runs per TMA row
      const double score = vol - 1e-3 * a - 1e-6 * b;
      if (score < best) {
        best = score;
        *tw = a; *th = b; *tb = c;
      }
    }
}

// Shared memory left for the operand ring after the epilogue's staging blocks and the control block.
static int ring_budget(int epi) {
  const int out_stg_bytes = (epi == EPI_PART) ? 0 : EPI_WARPS * HB_BYTES;
  const int fixed = out_stg_bytes + (epi == EPI_DX ? EPI_WARPS * HB_BYTES : 0) + static_cast<int>(sizeof(SmemCtl)) +
                    (epi == EPI_FWD ? EPI_WARPS * 384 * 4 : 0);
  return 227 * 1024 - 1024 - fixed;
}

// Column-sharing tiles (see GemmParams::colshare): one image per box and a box width that is a
// multiple of 8 pixels, so that a shift by one pixel row moves the operand by whole swizzle
// atoms.  Returns false when every such box wastes more than 15 % of its pixels on this extent.
bool conv_colshare_box(int W, int H, int rows_extra, int* tw, int* th) {
  double best = 1e300;
  bool found = false;
  // (32 x 4 boxes were measured too: with so few rows per box the shared box saves too little)
  const int cand[2][2] = {{8, 16}, {16, 8}};
  for (int i = 0; i < 2; ++i) {
    const int a = cand[i][0], b = cand[i][1];
    const double vol = static_cast<double>(ceil_div(W, a) * a) * static_cast<double>(ceil_div(H, b) * b);
    if (vol > 1.15 * W * H) continue;
    // at equal waste, the box that loads the fewest halo rows
    const double score = vol * (1.0 + 1e-3 * (b + rows_extra) / b);
    if (score < best) {
      best = score;
      *tw = a; *th = b;
      found = true;
    }
  }
  return found;
}

// Tile width for the forward / grad-input GEMMs: multiples of 64 so that every 128-byte
// staging row of the epilogue lies inside one tile.
static int choose_bn(int64_t Mr, int64_t Nc, int sm_count) {
  if (Nc <= 64) return 64;
  const int64_t mt = ceil_div(Mr, BM);
  int best = 64;
  double best_cost = 1e300;
  for (int bn = 256; bn >= 64; bn -= 64) {
    const int64_t tiles = mt * ceil_div(Nc, bn);
    const double cost = static_cast<double>(ceil_div(tiles, sm_count)) * (bn + 24);
    if (cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

int gemm_dx_num_partials(int64_t Mr, int64_t Nc) {
  // upper bound over every tile width the heuristic may pick: 8 epilogue warps per 128-row tile
  return static_cast<int>(ceil_div(Mr, BM) * ceil_div(Nc, 64) * EPI_WARPS);
}

static int part_bn(int64_t Nc) {
  return (Nc <= 64) ? static_cast<int>(round_up(Nc, 16)) : (Nc <= 128 ? 128 : 256);
}

int64_t gemm_part_tiles(int64_t Mr, int64_t Nc) { return ceil_div(Mr, BM) * ceil_div(Nc, part_bn(Nc)); }

int gemm_choose_splits(int64_t Mr, int64_t Nc, int64_t Kc, int sm_count) {
  const int64_t nkb = ceil_div(Kc, BK);
  const int64_t tiles = ceil_div(Mr, BM) * ceil_div(Nc, part_bn(Nc));
  int64_t max_s = nkb / 4 > 0 ? nkb / 4 : 1;        // at least four contraction blocks per split
  // More tiles than SMs: a short last wave can cost up to half a tile time, and splitting the
  // contraction in 2-4 makes the work items smaller.  Fewer tiles than SMs: split until the SMs
  // are full, but never into a second, nearly empty wave (32 tiles x 5 splits = 160 items on 148
  // SMs took twice the time of 32 x 4).  Either way: the split with the fewest tile times,
  // charging 2 % per extra split for the larger partial-product traffic.
  if (tiles >= sm_count && max_s > 4) max_s = 4;
  if (max_s > sm_count) max_s = sm_count;
  int best = 1;
  double best_cost = 1e300;
  for (int64_t c = 1; c <= max_s; ++c) {
    const double cost = static_cast<double>(ceil_div(tiles * c, sm_count)) / c * (1.0 + 0.02 * (c - 1));
    if (cost < best_cost - 1e-12) {
      best_cost = cost;
      best = static_cast<int>(c);
    }
    if (tiles * c > 2 * static_cast<int64_t>(sm_count) && tiles < sm_count) break;
  }
  return best;
}

template <int A_MN, int B_MN, int EPI, int CTA2>
static int launch(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to, const CUtensorMap& tx,
                  const CUtensorMap* tcls, const GemmParams& p, int grid, size_t smem, cudaStream_t st) {
  auto kern = gemm_kernel<A_MN, B_MN, EPI, CTA2>;
  count_launches(1);
  if (launch_dependent(kern, static_cast<unsigned>(grid), GEMM_THREADS, smem, st, CTA2 ? 2 : 1, ta, tb, to, tx,
                       tcls[0], tcls[1], tcls[2], p) != cudaSuccess)
    return EFQAT_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
}

template <int A_MN, int B_MN, int EPI, int CTA2>
static bool allow_full_smem() {
  return cudaFuncSetAttribute(gemm_kernel<A_MN, B_MN, EPI, CTA2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              227 * 1024) == cudaSuccess;
}

// Per device, with that device current (efqat_create): every instantiation of the kernel may
// use the whole shared memory of an SM.
int gemm_init() {
  if (!tensor_map_encoder()) return EFQAT_ERR_CUDA;
  const bool ok = allow_full_smem<0, 0, EPI_FWD, 0>() && allow_full_smem<0, 0, EPI_FWD, 1>() &&
                  allow_full_smem<0, 0, EPI_FWD_I8, 0>() && allow_full_smem<0, 0, EPI_FWD_I8, 1>() &&
                  allow_full_smem<0, 1, EPI_DX, 0>() && allow_full_smem<0, 1, EPI_DX, 1>() &&
                  allow_full_smem<1, 1, EPI_PART, 0>() && allow_full_smem<1, 1, EPI_PART, 1>() &&
                  allow_full_smem<0, 0, EPI_PART, 0>() && allow_full_smem<0, 1, EPI_PART, 0>() &&
                  allow_full_smem<1, 0, EPI_PART, 0>();
  return ok ? EFQAT_OK : EFQAT_ERR_CUDA;
}

int run_gemm(const GemmArgs& a, int sm_count, cudaStream_t st, int* tiles_out, int* grid_out) {
  if (a.Mr < 1 || a.Nc < 1 || a.Kc < 1) return EFQAT_ERR_SHAPE;
  int rc = EFQAT_OK;
  GemmParams p = {};
  p.Mr = a.Mr;
  p.Nc = a.Nc;
  // forward of a plain layer on integer operands: 8-bit codes, 128 of them per 128-byte k-block
  const int i8 = (a.epi == EPI_FWD && a.i8 && !a.conv && !a.a_mn && !a.b_mn) ? 1 : 0;
  p.i8 = i8;
  p.bk = i8 ? 128 : BK;
  p.a_signed = a.x_sym ? 1 : 0;
  p.wsum = a.wsum;
  p.nkb = static_cast<int>(ceil_div(a.Kc, p.bk));
  p.splits = (a.epi == EPI_PART) ? a.splits : 1;
  if (p.splits < 1 || p.splits > p.nkb) return EFQAT_ERR_SHAPE;
  p.BN = (a.epi == EPI_PART) ? part_bn(a.Nc) : choose_bn(a.Mr, a.Nc, sm_count);
  const ConvArgs* cv = a.conv;
  const int cs = cv ? cv->stride : 1;           // convolution stride
  int cWc = 0, cHc = 0;                         // grad-input: extent of this launch's pixel class
  ConvP col_taps = {};                          // the taps re-ordered (and filled up) for column sharing
  if (cv) {
    if (cv->mode < 1 || cv->mode > 3 || cs < 1 || cs > 2 || cv->R * cv->S > MAX_TAPS) return EFQAT_ERR_UNIMPL;
    if (cv->mode == 2) {           // grad-input tiles must not straddle the end of Cin (B is not zero there)
      const int64_t ncols = cv->ex ? a.Nc : cv->Cin;
      p.BN = (ncols % 256 == 0) ? 256 : (ncols % 192 == 0) ? 192 : (ncols % 128 == 0) ? 128 : 64;
      if (cv->ex) {
        cWc = cv->ex->pW;
        cHc = cv->ex->pH;
      } else {
        if (cv->cls_h < 0 || cv->cls_h >= cs || cv->cls_w < 0 || cv->cls_w >= cs) return EFQAT_ERR_SHAPE;
        cWc = static_cast<int>(ceil_div(cv->W - cv->cls_w, cs));
        cHc = static_cast<int>(ceil_div(cv->H - cv->cls_h, cs));
      }
    }
    // filter taps of this launch
    ConvP& c = p.cv;
    c.ntaps = 0;
    if (cv->mode == 2 && cv->ex) {
      const ConvExplicit& ex = *cv->ex;
      if (ex.ntaps < 0 || ex.ntaps > MAX_TAPS) return EFQAT_ERR_SHAPE;
      c.ntaps = ex.ntaps;
      for (int t = 0; t < ex.ntaps; ++t) {
        c.tap_dh[t] = ex.tap_dh[t]; c.tap_dw[t] = ex.tap_dw[t];
        c.tap_map[t] = ex.tap_map[t]; c.tap_rs[t] = ex.tap_rs[t];
      }
    } else
    for (int r = 0; r < cv->R; ++r)
      for (int sx = 0; sx < cv->S; ++sx) {
        int dh, dw, mi = 0;
        if (cv->mode == 2) {
          // input pixel h = cls_h + stride * i receives tap r from output row (h + pad - r) / stride
          const int nh = cv->cls_h + cv->pad - r, nw = cv->cls_w + cv->pad - sx;
          if (nh % cs != 0 || nw % cs != 0) continue;
          dh = nh / cs;
          dw = nw / cs;
        } else {
          // output pixel ho reads input row stride * ho + r - pad = stride * (ho + dh) + class
          const int oh = r - cv->pad, ow = sx - cv->pad;
          const int ah = ((oh % cs) + cs) % cs, aw = ((ow % cs) + cs) % cs;
          dh = (oh - ah) / cs;
          dw = (ow - aw) / cs;
          mi = ah * cs + aw;
        }
        c.tap_dh[c.ntaps] = static_cast<int8_t>(dh);
        c.tap_dw[c.ntaps] = static_cast<int8_t>(dw);
        c.tap_map[c.ntaps] = static_cast<uint8_t>(mi);
        c.tap_rs[c.ntaps] = static_cast<uint8_t>(r * cv->S + sx);
        ++c.ntaps;
      }
    if (c.ntaps == 0 || (cv->mode == 2 && (cWc < 1 || cHc < 1))) {     // nothing reaches this pixel class
      if (tiles_out) *tiles_out = 0;
      if (grid_out) *grid_out = 0;
      return EFQAT_OK;
    }
    // Column sharing: the taps must form groups, each with one tensor map, one dw and consecutive
    // dh (the rows of one filter column); they are then re-ordered group by group, smallest row
    // shift first.  Groups of unequal size (a strided forward reads even and odd filter rows
    // through different maps) are filled up with taps whose weight columns lie past the end of the
    // weight matrix, i.e. read as zeros, as long as that adds at most 15 % of blocks.
    if ((cv->mode == 2 || cv->mode == 1) && c.ntaps >= 2) {
      int order[MAX_TAPS], n = c.ntaps, gmax = 0, groups = 0;
      for (int j = 0; j < n; ++j) order[j] = j;
      for (int i = 1; i < n; ++i)                         // insertion sort by (map, dw, dh)
        for (int j = i; j > 0; --j) {
          const int x = order[j - 1], y = order[j];
          const int kx = c.tap_map[x] * 256 + c.tap_dw[x], ky = c.tap_map[y] * 256 + c.tap_dw[y];
          if (kx < ky || (kx == ky && c.tap_dh[x] <= c.tap_dh[y])) break;
          order[j - 1] = y; order[j] = x;
        }
      bool grid = true;
      for (int first = 0; first < n && grid;) {
        int last = first + 1;
        while (last < n && c.tap_dw[order[last]] == c.tap_dw[order[first]] &&
               c.tap_map[order[last]] == c.tap_map[order[first]]) ++last;
        if (last - first > gmax) gmax = last - first;
        ++groups;
        for (int j = first + 1; j < last && grid; ++j)
          if (c.tap_dh[order[j]] != c.tap_dh[order[j - 1]] + 1) grid = false;
        first = last;
      }
      const int padded = groups * gmax;
      const bool may_pad = cv->mode == 1 && !a.b_mn && cv->R * cv->S < 255;
      if (grid && gmax >= 2 && gmax <= 4 && padded <= MAX_TAPS &&
          (padded == n || (may_pad && padded * 20 <= n * 23))) {
        p.colshare = gmax;
        col_taps = c;
        int m = 0;
        for (int first = 0; first < n;) {
          int last = first + 1;
          while (last < n && c.tap_dw[order[last]] == c.tap_dw[order[first]] &&
                 c.tap_map[order[last]] == c.tap_map[order[first]]) ++last;
          for (int j = 0; j < gmax; ++j, ++m) {
            const int src = order[first + j < last ? first + j : last - 1];
            col_taps.tap_dh[m] = static_cast<int8_t>(c.tap_dh[order[first]] + j);
            col_taps.tap_dw[m] = c.tap_dw[src];
            col_taps.tap_map[m] = c.tap_map[src];
            col_taps.tap_rs[m] = first + j < last ? c.tap_rs[src] : static_cast<uint8_t>(cv->R * cv->S);
          }
          first = last;
        }
        col_taps.ntaps = m;
      }
    }
  }
  // CTA pairs (256 x BN tiles, tiles full in N) halve the B traffic from L2 per FLOP; they are
  // taken unless one-CTA tiles fill the machine's last wave clearly better.
  int pair = 0;
  // Full weight-gradient GEMM (both operands MN-major), as measured at M = 16384 over ten (K, N)
  // shapes: pairs give 1.22-1.43 PFLOP/s against 1.0-1.17 for one-CTA tiles, except on the two
  // squares 4096^2 and 5120^2 (0.88-0.96 against 1.09-1.12), for which no cause was found.
  // Pairs are therefore taken when the smaller output extent is at most 3072 and there are at
  // least 64 pair tiles (small problems, split many ways, lose: 768^2 went from 24 to 39 us),
  // or on long runs (>= 512, the shortest measured good one) of unsplit pair tiles.
  const int64_t pair_tiles = ceil_div(a.Mr, 2 * BM) * (a.Nc / 256);
  const int64_t small_ext = a.Mr < a.Nc ? a.Mr : a.Nc;
  const bool part_pair = a.a_mn && a.b_mn && a.Nc % 256 == 0 &&
                         ((a.splits == 1 && pair_tiles >= 512) ||
                          (small_ext <= 3072 && pair_tiles >= 64));
  if (!cv && (a.epi != EPI_PART || part_pair) && a.Mr >= 256 && a.Nc % 128 == 0) {
    const int units = sm_count / 2;
    const int64_t mt = ceil_div(a.Mr, 2 * BM);
    const bool can256 = a.Nc % 256 == 0;
    const double c256 = can256 ? static_cast<double>(ceil_div(mt * (a.Nc / 256), units)) * (256 + 24) : 1e300;
    const double c128 = static_cast<double>(ceil_div(mt * (a.Nc / 128), units)) * (128 + 24);
    const int bn_pair = (c256 <= c128) ? 256 : 128;
    const double c_pair = 0.92 * (c256 <= c128 ? c256 : c128);
    const double c_single = static_cast<double>(ceil_div(ceil_div(a.Mr, BM) * ceil_div(a.Nc, p.BN), sm_count)) * (p.BN + 24);
    if (c_pair <= c_single) {
      pair = 1;
      p.BN = bn_pair;
    }
  }
  const int bn_cta = pair ? p.BN / 2 : p.BN;
  p.tiles_m = static_cast<int>(ceil_div(a.Mr, pair ? 2 * BM : BM));
  p.tiles_n = static_cast<int>(ceil_div(a.Nc, p.BN));
  if (cv) {
    ConvP& c = p.cv;
    c.mode = cv->mode;
    // pixel space that is tiled: outputs for forward and grad-weight, the launch's class of
    // input pixels for grad-input
    const int pW = (cv->mode == 2) ? cWc : cv->Wo, pH = (cv->mode == 2) ? cHc : cv->Ho;
    conv_pixel_box(pW, pH, cv->B, cv->mode == 3 ? BK : BM, &c.tw, &c.th, &c.tb);
    if (p.colshare) {
      // taken when a suitable box exists and two stages (with the B operand resident or staged) fit
      int tw2 = 0, th2 = 0;
      bool fits = conv_colshare_box(pW, pH, p.colshare - 1, &tw2, &th2);
      if (fits) {
        const int a_reg = static_cast<int>(round_up((th2 + p.colshare - 1) * tw2 * 128, 1024));
        const int b_st = static_cast<int>(round_up(a.b_mn ? ceil_div(bn_cta, 64) * CHUNK_BYTES : bn_cta * BK * 2, 1024));
        const int nkb2 = col_taps.ntaps * static_cast<int>(ceil_div((cv->mode == 2) ? cv->N : cv->Cin, 64));
        const int ring = ring_budget(a.epi);
        const bool res = p.tiles_n == 1 && static_cast<int64_t>(nkb2) * b_st + 2 * a_reg <= ring;
        fits = res || ring / (a_reg + p.colshare * b_st) >= 2;
        if (fits) {
          c.tw = tw2; c.th = th2; c.tb = 1;
          p.bres = res ? 1 : 0;
          p.a_region_bytes = a_reg;
          p.a_tx = (th2 + p.colshare - 1) * tw2 * 128;
          c.ntaps = col_taps.ntaps;
          for (int j = 0; j < c.ntaps; ++j) {
            c.tap_dh[j] = col_taps.tap_dh[j]; c.tap_dw[j] = col_taps.tap_dw[j];
            c.tap_map[j] = col_taps.tap_map[j]; c.tap_rs[j] = col_taps.tap_rs[j];
          }
        }
      }
      if (!fits) p.colshare = 0;
    }
    c.tiles_w = static_cast<int>(ceil_div(pW, c.tw));
    c.tiles_h = static_cast<int>(ceil_div(pH, c.th));
    const int tiles_b = static_cast<int>(ceil_div(cv->B, c.tb));
    c.dimH = pH; c.dimB = cv->B;
    c.C = (cv->mode == 2) ? cv->N : cv->Cin;
    c.cchunks = static_cast<int>(ceil_div(c.C, 64));
    c.wcols = (cv->mode == 2 && cv->ex) ? 64 : cv->Cin;
    if (cv->mode == 3) {
      p.nkb = c.tiles_w * c.tiles_h * tiles_b;                 // contraction over boxes of 64 output pixels
      if (p.splits > p.nkb) return EFQAT_ERR_SHAPE;
      p.tiles_m = static_cast<int>(ceil_div(static_cast<int64_t>(c.ntaps) * c.cchunks * 64, BM));   // rows = (tap, padded channel)
    } else {
      p.tiles_m = c.tiles_w * c.tiles_h * tiles_b;             // one tile per box of 128 pixels
      p.nkb = c.ntaps * c.cchunks;
    }
  }
  // Order of the work list.  One tile reads tile_rows x Kc of A and BN x Kc of B.  With the
  // plain row-major order the tiles in flight sweep every tile column, i.e. all of B, once per
  // wave; when B is larger than what L2 keeps, each wave fetches it from DRAM again (measured
  // on M = 16384, 8192 x 8192: 5.6 GB read for 0.67 GB of operands).  Panels sized to about
  // L2_PANEL_BYTES keep one operand's slice resident while the other streams past it once per
  // panel; the direction with the smaller estimated DRAM traffic wins, and plain order stays
  // when a whole operand fits the panel budget anyway.
  {
    const double es = i8 ? 1.0 : 2.0;
    const double kc_bytes = static_cast<double>(p.nkb) * p.bk * es / (p.splits > 0 ? p.splits : 1);
    const double a_tile = static_cast<double>(pair ? 2 * BM : BM) * kc_bytes;
    const double b_tile = static_cast<double>(p.BN) * kc_bytes;
    const double a_all = a_tile * p.tiles_m, b_all = b_tile * p.tiles_n;
    p.panel_dir = 0;
    p.panel = 0;
    if (b_all > L2_PANEL_BYTES && a_all > L2_PANEL_BYTES && p.tiles_m > 1 && p.tiles_n > 1) {
      int gn = static_cast<int>(L2_PANEL_BYTES / b_tile), gm = static_cast<int>(L2_PANEL_BYTES / a_tile);
      if (gn < 1) gn = 1;
      if (gm < 1) gm = 1;
      const double t_n = a_all * static_cast<double>(ceil_div(p.tiles_n, gn)) + b_all;   // column panels
      const double t_m = b_all * static_cast<double>(ceil_div(p.tiles_m, gm)) + a_all;   // row panels
      if (t_n <= t_m) { p.panel_dir = 1; p.panel = gn; } else { p.panel_dir = 2; p.panel = gm; }
    }
    // The panel's operand is asked to stay (L2 evict-last) while the other one streams past with
    // the normal policy.  Measured on M = 16384, 8192 x 8192 and 4096 x 16384 (grad-input GEMM):
    // 1.31 -> 1.32 PFLOP/s; marking the streamed operand evict-first costs 5-14 % (a row block is
    // read by the `panel` tiles of its row at slightly different times), and panels of 16, 24 or
    // 48 MB instead of 32 are 10-20 % slower.
    if (p.panel_dir == 1) p.hint_b = 2;
    else if (p.panel_dir == 2) p.hint_a = 2;
  }
  p.blk_cols = a.out_bf16 ? 32 : 16;
  p.b_stage_bytes = static_cast<int>(a.b_mn ? ceil_div(bn_cta, 64) * CHUNK_BYTES : bn_cta * BK * 2);
  p.b_stage_bytes = static_cast<int>(round_up(p.b_stage_bytes, 1024));
  const int sub_bytes = A_STAGE_BYTES + p.b_stage_bytes;
  const int out_stg_bytes = (a.epi == EPI_PART) ? 0 : EPI_WARPS * HB_BYTES;     // one staging buffer per warp
  int fixed_bytes = 227 * 1024 - 1024 - ring_budget(a.epi);
  int ring_bytes = ring_budget(a.epi);
  // k-blocks per stage: as many as still leave three stages (two for the widest tiles), at most 4
  int kps = ring_bytes / (3 * sub_bytes);
  if (kps <= 1) kps = (ring_bytes / (2 * sub_bytes) >= 2) ? 2 : 1;
  if (kps > 4) kps = 4;
  if (kps > p.nkb) kps = p.nkb;
  int bres_bytes = 0;
  if (p.colshare) {
    kps = p.colshare;
    p.a_sub_off = p.cv.tw * 128;
    p.b_region_bytes = p.bres ? 0 : kps * p.b_stage_bytes;
    bres_bytes = p.bres ? p.nkb * p.b_stage_bytes : 0;
    ring_bytes -= bres_bytes;
  } else {
    p.a_region_bytes = kps * A_STAGE_BYTES;
    p.b_region_bytes = kps * p.b_stage_bytes;
    p.a_sub_off = A_STAGE_BYTES;
  }
  p.kps = kps;
  p.merged = cv ? 0 : 1;
  const int stage_bytes = p.a_region_bytes + p.b_region_bytes;
  int stages = ring_bytes / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return EFQAT_ERR_SHAPE;
  p.stages = stages;
  // a second staging buffer per epilogue warp when the ring leaves room for it
  p.out_bufs = 1;
  if (out_stg_bytes && ring_bytes - stages * stage_bytes >= out_stg_bytes) {
    p.out_bufs = 2;
    fixed_bytes += out_stg_bytes;
  }
  p.col_scale = a.col_scale;
  p.col_bias = a.col_bias;
  p.s_x = a.s_x; p.z_x = a.z_x; p.x_bits = a.x_bits; p.x_sym = a.x_sym;
  p.partials = a.partials;
  p.out = static_cast<float*>(a.out);
  p.ldo = a.ldo;
  p.split_stride = a.split_stride;
  p.part_cols = a.part_cols;
  p.status = a.status;
  p.defer_wait = a.defer_wait;

  CUtensorMap ta, tb, to, tx, tcls[3];
  if (a.epi == EPI_DX && (a.x_dtype == EFQAT_BF16) != (a.out_bf16 != 0)) return EFQAT_ERR_DTYPE;
  if (!cv) {
    // MN-major operands: one box = all kps k-blocks of a stage for one 64-wide chunk
    rc = a.a_mn ? make_map(&ta, a.A, 1, a.Kc, a.Mr, a.lda, BK * kps) : make_map(&ta, a.A, i8 ? 2 : 1, a.Mr, a.Kc, a.lda, BM);
    if (rc != EFQAT_OK) return rc;
    rc = a.b_mn ? make_map(&tb, a.B, 1, a.Kc, a.Nc, a.ldb, BK * kps) : make_map(&tb, a.B, i8 ? 2 : 1, a.Nc, a.Kc, a.ldb, bn_cta);
    if (rc != EFQAT_OK) return rc;
    to = ta;
    tx = ta;
    tcls[0] = tcls[1] = tcls[2] = ta;
    if (a.epi != EPI_PART) {
      rc = make_map(&to, a.out, a.out_bf16, a.Mr, a.Nc, a.ldo, 32, 64);
      if (rc != EFQAT_OK) return rc;
    }
    if (a.epi == EPI_DX) {
      rc = make_map(&tx, a.X, a.out_bf16, a.Mr, a.Nc, a.ldo, 32, 64);
      if (rc != EFQAT_OK) return rc;
    }
  } else {
    const ConvP& c = p.cv;
    const int64_t KK = (cv->mode == 2 && cv->ex) ? cv->ex->b_cols : static_cast<int64_t>(cv->R) * cv->S * cv->Cin;
    // quarter of a 128-pixel box: the 32 rows one epilogue warp owns
    const int qh = (32 / c.tw < c.th) ? 32 / c.tw : c.th;
    const int qb = 32 / (c.tw * qh);
    // The input activation tensor seen as stride x stride interleaved sub-grids of pixels: class
    // (ah, aw) holds the pixels (ah + stride * i, aw + stride * j).
    const int64_t Ci = cv->Cin, HW = static_cast<int64_t>(cv->H) * cv->W;
    auto class_map = [&](CUtensorMap* m, const void* base, int is16, int ah, int aw, int bw_, int bh_, int bb_,
                         int row_bytes, int64_t ppix = 0, int64_t prow = 0, int64_t pimg = 0) {
      if (!ppix) ppix = Ci;
      if (!prow) prow = cv->W * Ci;
      if (!pimg) pimg = Ci * HW;
      const int64_t Wc = ceil_div(cv->W - aw, cs), Hc = ceil_div(cv->H - ah, cs);
      if (Wc < 1 || Hc < 1) return make_map_4d(m, base, is16, cv->B, 1, 1, Ci, Ci, bw_, bh_, bb_, row_bytes, ppix, prow,
                                               pimg);        // empty class: never addressed by a tap
      const char* b0 = static_cast<const char*>(base) + (static_cast<int64_t>(ah) * prow + aw * ppix) * (is16 ? 2 : 4);
      return make_map_4d(m, b0, is16, cv->B, Hc, Wc, Ci, Ci, bw_, bh_, bb_, row_bytes, cs * ppix, cs * prow, pimg);
    };
    if (cv->mode == 1 || cv->mode == 3) {
      CUtensorMap* maps[4] = {&ta, &tcls[0], &tcls[1], &tcls[2]};
      for (int i = 0; i < 4 && rc == EFQAT_OK; ++i) {
        const int ah = (i < cs * cs) ? i / cs : 0, aw = (i < cs * cs) ? i % cs : 0;
        rc = class_map(maps[i], a.A, 1, ah, aw, c.tw, c.th + (p.colshare ? p.colshare - 1 : 0), c.tb, 128, cv->pix_pitch,
                       cv->row_pitch, cv->img_pitch);
      }
    }
    if (cv->mode == 1) {
      if (rc == EFQAT_OK) rc = make_map(&tb, a.B, 1, cv->N, KK, KK, bn_cta);
      if (rc == EFQAT_OK)
        rc = make_map_4d(&to, a.out, a.out_bf16, cv->B, cv->Ho, cv->Wo, cv->N, cv->N, c.tw, qh, qb, 64);
      tx = ta;
    } else if (cv->mode == 2 && cv->ex) {
      const ConvExplicit& ex = *cv->ex;
      CUtensorMap* maps[4] = {&ta, &tcls[0], &tcls[1], &tcls[2]};
      for (int i = 0; i < 4 && rc == EFQAT_OK; ++i) {
        const ConvView& v = ex.a_view[ex.a_view[i].base ? i : 0];
        rc = make_map_4d(maps[i], v.base, 1, cv->B, v.H, v.W, cv->N, cv->N, c.tw, c.th + (p.colshare ? p.colshare - 1 : 0),
                         c.tb, 128, v.pix, v.row, v.img);
      }
      if (rc == EFQAT_OK) rc = make_map(&tb, a.B, 1, cv->N, KK, KK, BK);
      const ConvView& o = ex.o_view;
      if (rc == EFQAT_OK)
        rc = make_map_4d(&to, o.base, a.out_bf16, cv->B, o.H, o.W, a.Nc, a.Nc, c.tw, qh, qb, 64, o.pix, o.row, o.img);
      if (rc == EFQAT_OK)
        rc = make_map_4d(&tx, ex.x_base, a.out_bf16, cv->B, o.H, o.W, a.Nc, a.Nc, c.tw, qh, qb, 64, o.pix, o.row, o.img);
    } else if (cv->mode == 2) {
      rc = make_map_4d(&ta, a.A, 1, cv->B, cv->Ho, cv->Wo, cv->N, cv->N, c.tw, c.th + (p.colshare ? p.colshare - 1 : 0), c.tb);
      tcls[0] = tcls[1] = tcls[2] = ta;
      if (rc == EFQAT_OK) rc = make_map(&tb, a.B, 1, cv->N, KK, KK, BK);
      if (rc == EFQAT_OK) rc = class_map(&to, a.out, a.out_bf16, cv->cls_h, cv->cls_w, c.tw, qh, qb, 64);
      if (rc == EFQAT_OK) rc = class_map(&tx, a.X, a.out_bf16, cv->cls_h, cv->cls_w, c.tw, qh, qb, 64);
    } else {
      if (rc == EFQAT_OK) rc = make_map_4d(&tb, a.B, 1, cv->B, cv->Ho, cv->Wo, a.Nc, a.ldb, c.tw, c.th, c.tb);
      to = ta;
      tx = ta;
    }
    if (rc != EFQAT_OK) return rc;
  }

  const int64_t items = static_cast<int64_t>(p.tiles_m) * p.tiles_n * p.splits;
  const int max_units = pair ? sm_count / 2 : sm_count;
  const int units = static_cast<int>(items < max_units ? items : max_units);
  const int grid = pair ? 2 * units : units;
  const size_t smem = static_cast<size_t>(stages) * stage_bytes + bres_bytes + fixed_bytes + 1024;
  // the (dS_x, dZ_x) pairs this launch writes must fit what the caller set aside for them
  if (a.epi == EPI_DX && a.partials_cap > 0 &&
      static_cast<int64_t>(p.tiles_m) * p.tiles_n * (pair ? 2 : 1) * EPI_WARPS > a.partials_cap)
    return EFQAT_ERR_WORKSPACE;
  if (tiles_out) *tiles_out = p.tiles_m * p.tiles_n * (pair ? 2 : 1) * EPI_WARPS;
  if (grid_out) *grid_out = grid;

#define EFQAT_LAUNCH(AM, BMj, E, P2) return launch<AM, BMj, E, P2>(ta, tb, to, tx, tcls, p, grid, smem, st)
  if (a.epi == EPI_FWD && !a.a_mn && !a.b_mn) {
    if (i8) {
      if (pair) EFQAT_LAUNCH(0, 0, EPI_FWD_I8, 1);
      EFQAT_LAUNCH(0, 0, EPI_FWD_I8, 0);
    }
    if (pair) EFQAT_LAUNCH(0, 0, EPI_FWD, 1);
    EFQAT_LAUNCH(0, 0, EPI_FWD, 0);
  }
  if (a.epi == EPI_DX && !a.a_mn && a.b_mn) {
    if (pair) EFQAT_LAUNCH(0, 1, EPI_DX, 1);
    EFQAT_LAUNCH(0, 1, EPI_DX, 0);
  }
  if (a.epi == EPI_PART && a.a_mn && a.b_mn) {
    if (pair) EFQAT_LAUNCH(1, 1, EPI_PART, 1);
    EFQAT_LAUNCH(1, 1, EPI_PART, 0);
  }
  if (a.epi == EPI_PART && !a.a_mn && !a.b_mn) EFQAT_LAUNCH(0, 0, EPI_PART, 0);
  if (a.epi == EPI_PART && !a.a_mn && a.b_mn) EFQAT_LAUNCH(0, 1, EPI_PART, 0);
  if (a.epi == EPI_PART && a.a_mn && !a.b_mn) EFQAT_LAUNCH(1, 0, EPI_PART, 0);
#undef EFQAT_LAUNCH
  return EFQAT_ERR_UNIMPL;
}

}  // namespace efqat
