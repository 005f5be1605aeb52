// Backward of layers with a contraction of 64 (the 1x1 convolutions of the first ResNet stage,
// 64 -> 128 / 256 channels) in ONE pass over dY and X.  These layers move more than a byte per
// 50 flop: HBM traffic bounds them, and the general path reads dY three times (column sums and
// gather, grad-input GEMM, gathered copy in the weight-gradient GEMM) and X twice.  Here a tile of
// 128 rows of dY is brought into shared memory once and feeds everything (Algorithm 1, Eq. 5):
//   * grad-input:  D1[m, k] = sum_n dY[m, n] W^[n, k]      (the tile as K-major A operand),
//   * weight grad: D2[n, k] = sum_m dY[m, n] (q_x[m, k] - Z) (the SAME bytes as MN-major A operand:
//     rows of the tile are the contraction index now), accumulated in TMEM over all tiles of the CTA,
//   * bias grad:   a column of ones appended to the activation-code operand makes D2[n, 64] the
//     column sum of dY,
// while the eight worker warps quantize X (Eq. 1) straight into the operand tile of the second
// MMA and run the straight-through epilogue of D1 (clip mask, dS_x / dZ_x partial sums) on the raw
// activations they kept in registers.  The weight gradient is computed for every channel of the
// tile -- with dY on chip the tensor pipe has the time, the layer being bound by bytes -- and only
// the rows of the unfrozen channels leave the SM, as one partial product per CTA that the finalize
// launch sums.  No gather, no code matrix, no second read of anything.
//
// Persistent, one CTA per SM, 320 threads: warp 0 TMA producer (ring of half tiles of dY, the X
// tile), warp 1 issues tcgen05.mma and owns TMEM, warps 2..9 workers.
#include "internal.h"
#include "ptx.cuh"

namespace efqat {

using namespace ptx;

namespace {

const int SB_THREADS = 320;
const int SB_ROWS = 128;                       // rows per tile = UMMA M of the grad-input product
const int SB_STAGES = 3;                       // half tiles of dY in flight
const int T16K = SB_ROWS * 128;                // [128 rows x 128 bytes]: one 64-column box of bf16
const int HALF_BYTES = 2 * T16K;               // half tile of dY: 128 rows x 128 columns
const int SB_WORKERS = 8;
const int D2_COL0 = 128, D2_STRIDE = 96;       // TMEM columns: D1 buffers at 0 and 64, D2 halves from 128
const int D2_N = 80;                           // 64 fan-in columns + the ones column, rounded to the MMA's N step

struct SkinnyBwdArgs {
  int64_t M;
  int N, nh, tiles;                            // nh = N / 128 half tiles per tile
  const float* W; const bf16* what; const float* s_w; int w_bits;
  const float* s_x; const float* z_x; int x_bits, x_sym;
  const int32_t* idx; int k_sel;
  float* P;                                    // [grid][k_sel][64] raw sums  dY^T (q_x - Z)
  float* colsum;                               // [grid][N] or null
  float* dxpart;                               // [grid * 8][2]
  int* status;
};

struct __align__(16) SbCtl {
  uint64_t full[SB_STAGES], empty[SB_STAGES];
  uint64_t x_full, x_empty;
  uint64_t xc_full[2], xc_empty[2];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t d2_full, drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint32_t sw128(int r, int j) { return r * 128 + ((j ^ (r & 7)) << 4); }
__device__ __forceinline__ uint8_t* stg64(uint8_t* base, int row, int piece) {
  return base + row * 64 + ((piece ^ ((row >> 1) & 3)) << 4);
}
__device__ __forceinline__ uint32_t pk2b(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__global__ void __launch_bounds__(SB_THREADS, 1)
skinny_bwd_kernel(const __grid_constant__ CUtensorMap tmDY, const __grid_constant__ CUtensorMap tmX,
                  const __grid_constant__ CUtensorMap tmDX, const SkinnyBwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* what_t = smem;                                // [N rows][128 B]: W^ as MN-major B of the grad-input MMA
  uint8_t* xc_t = what_t + a.N * 128;                    // [2][128 rows][128 B] centred activation codes
  uint8_t* ones_t = xc_t + 2 * T16K;                     // [128 rows][128 B]: column 0 = 1, rest 0
  uint8_t* xraw_t = ones_t + T16K;                       // [128 rows][128 B] raw X tile
  uint8_t* ring = xraw_t + T16K;                         // [SB_STAGES][2][128 rows][128 B]
  uint8_t* stg = ring + SB_STAGES * HALF_BYTES;          // [8 warps][2][32 rows][64 B]
  SbCtl* ctl = reinterpret_cast<SbCtl*>(stg + SB_WORKERS * 2 * 2048);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < SB_STAGES; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    mbar_init(&ctl->x_full, 1);
    mbar_init(&ctl->x_empty, SB_WORKERS);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->xc_full[b], SB_WORKERS);
      mbar_init(&ctl->xc_empty[b], 1);
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], SB_WORKERS);
    }
    mbar_init(&ctl->d2_full, 1);
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmDY);
    prefetch_tmap(&tmX);
    prefetch_tmap(&tmDX);
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, 512);
    tmem_relinquish();
  }
  pdl_trigger();
  pdl_wait();
  __syncthreads();                                       // barriers are initialised
  const int my_tiles = (a.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  // The first tile's copies need nothing of the set-up below: they travel while it runs.
  if (tid == 0 && my_tiles > 0) {
    const int t = blockIdx.x;
    mbar_arrive_expect_tx(&ctl->x_full, T16K);
    tma_load_2d(xraw_t, &tmX, &ctl->x_full, 0, t * SB_ROWS);
    for (int h = 0; h < a.nh; ++h) {
      mbar_arrive_expect_tx(&ctl->full[h], HALF_BYTES);
      tma_load_2d(ring + h * HALF_BYTES, &tmDY, &ctl->full[h], h * 128, t * SB_ROWS);
      tma_load_2d(ring + h * HALF_BYTES + T16K, &tmDY, &ctl->full[h], h * 128 + 64, t * SB_ROWS);
    }
  }

  // ---- resident operands: W^ = bf16(s_w q_w) (Eq. 3), one thread per channel with the whole row's
  // loads in flight at once (this phase is a chain of L2 round trips, not bandwidth), and the ones tile
  bool bad_scale = false;
  for (int n = tid - 32; n >= 0 && n < a.N; n += SB_THREADS - 32) {
    if (a.what) {
      uint4 o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = __ldg(reinterpret_cast<const uint4*>(a.what + static_cast<int64_t>(n) * 64) + j);
#pragma unroll
      for (int j = 0; j < 8; ++j) *reinterpret_cast<uint4*>(what_t + sw128(n, j)) = o[j];
    } else {
      float4 w4[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) w4[j] = __ldg(reinterpret_cast<const float4*>(a.W + static_cast<int64_t>(n) * 64) + j);
      float sw = __ldg(a.s_w + n);
      if (!scale_ok(sw)) {
        bad_scale = true;
        sw = 1.f;
      }
      const RowQ rq = make_rowq(sw, a.w_bits);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float w[8] = {w4[2 * j].x, w4[2 * j].y, w4[2 * j].z, w4[2 * j].w,
                            w4[2 * j + 1].x, w4[2 * j + 1].y, w4[2 * j + 1].z, w4[2 * j + 1].w};
        float d[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) d[i] = __fmul_rn(rq.s, quant_weight(w[i], rq).c0);
        *reinterpret_cast<uint4*>(what_t + sw128(n, j)) =
            make_uint4(pk2b(d[0], d[1]), pk2b(d[2], d[3]), pk2b(d[4], d[5]), pk2b(d[6], d[7]));
      }
    }
  }
  for (int p = tid; p < SB_ROWS * 8; p += SB_THREADS) {
    const int r = p >> 3, j = p & 7;
    *reinterpret_cast<uint4*>(ones_t + sw128(r, j)) = make_uint4(j == 0 ? 0x00003F80u : 0u, 0u, 0u, 0u);
  }
  bool bad_x;
  const ActQ xq = make_actq(a.s_x, a.z_x, a.x_bits, a.x_sym, &bad_x);
  if ((bad_scale || (bad_x && tid == 0)) && blockIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
  if (blockIdx.x == 0 && a.idx && a.k_sel < a.N) {       // index contract: inside [0, N), strictly ascending
    for (int i = tid; i < a.k_sel; i += SB_THREADS) {
      const int c = a.idx[i];
      if (c < 0 || c >= a.N || (i > 0 && a.idx[i - 1] >= c)) record_status(a.status, EFQAT_DEV_BAD_INDEX);
    }
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int it = a.nh;                                     // tile 0 was requested before the set-up
      bool live = true;
      for (int n = 1; n < my_tiles && live; ++n) {
        const int t = blockIdx.x + n * gridDim.x;
        if (*abort_flag || !mbar_wait(&ctl->x_empty, (n & 1) ^ 1)) { live = false; break; }
        mbar_arrive_expect_tx(&ctl->x_full, T16K);
        tma_load_2d(xraw_t, &tmX, &ctl->x_full, 0, t * SB_ROWS);
        for (int h = 0; h < a.nh; ++h, ++it) {
          const int s = it % SB_STAGES;
          if (*abort_flag || !mbar_wait(&ctl->empty[s], ((it / SB_STAGES) & 1) ^ 1)) { live = false; break; }
          mbar_arrive_expect_tx(&ctl->full[s], HALF_BYTES);
          tma_load_2d(ring + s * HALF_BYTES, &tmDY, &ctl->full[s], h * 128, t * SB_ROWS);
          tma_load_2d(ring + s * HALF_BYTES + T16K, &tmDY, &ctl->full[s], h * 128 + 64, t * SB_ROWS);
        }
      }
      if (!live) {
        record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
        *abort_flag = 1;
        // copies already issued must have landed before the CTA exits
        for (int j = (it > SB_STAGES ? it - SB_STAGES : 0); j < it; ++j)
          mbar_wait(&ctl->full[j % SB_STAGES], (j / SB_STAGES) & 1, 20000000ull);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = instr_desc_bf16(SB_ROWS, 64, 0, 1);        // dY (K-major) x W^ (MN-major)
      const uint32_t idesc2 = instr_desc_bf16(SB_ROWS, D2_N, 1, 1);      // dY^T (MN-major) x [codes | ones] (MN-major)
      const uint32_t what_addr = smem_u32(what_t), ones_addr = smem_u32(ones_t);
      int it = 0;
      bool ok = true;
      for (int n = 0; n < my_tiles && ok; ++n) {
        const int b = n & 1;
        if (*abort_flag || !mbar_wait(&ctl->acc_empty[b], ((n >> 1) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d1 = tmem_base + b * 64;
        const uint32_t xc_addr = smem_u32(xc_t + b * T16K);
        for (int h = 0; h < a.nh && ok; ++h, ++it) {
          const int s = it % SB_STAGES;
          if (*abort_flag || !mbar_wait(&ctl->full[s], (it / SB_STAGES) & 1)) { ok = false; break; }
          tc_fence_after();
          const uint32_t st_addr = smem_u32(ring + s * HALF_BYTES);
#pragma unroll
          for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16(d1, smem_desc_sw128(st_addr + j * T16K + k * 32, 16, 1024),
                        smem_desc_sw128(what_addr + (h * 128 + j * 64 + k * 16) * 128, 8192, 1024), idesc1,
                        (h | j | k) ? 1u : 0u);
          if (h == 0) {
            if (*abort_flag || !mbar_wait(&ctl->xc_full[b], (n >> 1) & 1)) { ok = false; break; }
            tc_fence_after();
          }
          const uint32_t d2 = tmem_base + D2_COL0 + h * D2_STRIDE;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_bf16(d2, smem_desc_sw128(st_addr + k * 2048, T16K, 1024),
                      smem_desc_sw128(xc_addr + k * 2048, ones_addr - xc_addr, 1024), idesc2, (n | k) ? 1u : 0u);
          umma_commit(&ctl->empty[s]);
        }
        if (ok) {
          umma_commit(&ctl->acc_full[b]);
          umma_commit(&ctl->xc_empty[b]);
        }
      }
      if (ok) {
        umma_commit(&ctl->d2_full);
      } else {
        record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
        *abort_flag = 1;
        umma_commit(&ctl->drain);
        mbar_wait(&ctl->drain, 0, 20000000ull);
      }
    }
  } else {
    // ------------------------------------------------------------- workers (warps 2..9)
    const int e = warp - 2, q = warp & 3, half = e >> 2;
    const int row = q * 32 + lane;                         // row of the tile this lane owns (quantizer and epilogue)
    uint8_t* my_stg = stg + e * 2 * 2048;
    const float c_lo = xq.lo - xq.zr, c_hi = xq.hi - xq.zr;
    const float t_lo = c_lo, t_hi = c_hi;                  // d/ds of a clipped element
    const float q_half = 0.5f * (xq.hi - xq.lo), z_mid = xq.zr - 0.5f * (xq.hi + xq.lo);
    float acc_s = 0.f, acc_c = 0.f;
    int st_it = 0;
    bool ok = true;

    // Eq. 1 on this lane's 32 values of tile number n: raw X from the staged tile (kept in xr for the
    // epilogue of the same tile), centred codes into operand buffer n & 1
    auto quant_tile = [&](int n, uint4 (&xr)[4]) -> bool {
      const int b = n & 1;
      bool g = *abort_flag ? false : mbar_wait(&ctl->x_full, n & 1);
      if (!__all_sync(0xffffffffu, g)) return false;
#pragma unroll
      for (int i = 0; i < 4; ++i) xr[i] = *reinterpret_cast<const uint4*>(xraw_t + sw128(row, half * 4 + i));
      fence_proxy_async();           // the next bulk copy into the raw tile is ordered behind these reads
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->x_empty);
      g = *abort_flag ? false : mbar_wait(&ctl->xc_empty[b], ((n >> 1) & 1) ^ 1);
      if (!__all_sync(0xffffffffu, g)) return false;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t wv[4] = {xr[i].x, xr[i].y, xr[i].z, xr[i].w};
        float c[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          c[2 * j] = __uint_as_float(wv[j] << 16);
          c[2 * j + 1] = __uint_as_float(wv[j] & 0xffff0000u);
        }
        // centred code: clamp(rne(x / s) + Zr, lo, hi) - Zr = clamp(rne(x / s), lo - Zr, hi - Zr) (integers, exact)
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = fminf(fmaxf(rne_small(__fmul_rn(c[j], xq.rinv)), c_lo), c_hi);
        *reinterpret_cast<uint4*>(xc_t + b * T16K + sw128(row, half * 4 + i)) =
            make_uint4(pk2b(c[0], c[1]), pk2b(c[2], c[3]), pk2b(c[4], c[5]), pk2b(c[6], c[7]));
      }
      fence_proxy_async();           // generic writes of the codes -> visible to the MMA's async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->xc_full[b]);
      return true;
    };

    uint4 xa[4], xb[4];
    if (my_tiles > 0) ok = quant_tile(0, xa);
    for (int n = 0; n < my_tiles && ok; ++n) {
      const int t = blockIdx.x + n * gridDim.x;
      const int b = n & 1;
      if (n + 1 < my_tiles) {
        ok = quant_tile(n + 1, xb);
        if (!ok) break;
      }
      bool g = *abort_flag ? false : mbar_wait(&ctl->acc_full[b], (n >> 1) & 1);
      if (!__all_sync(0xffffffffu, g)) { ok = false; break; }
      tc_fence_after();
      uint32_t r[32];
      tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 64 + half * 32, r);
      uint8_t* ob = my_stg + (st_it & 1) * 2048;
      ++st_it;
      if (lane == 0) tma_store_wait_read1();
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);      // the accumulator is in registers
#pragma unroll
      for (int gi = 0; gi < 4; ++gi) {
        const uint32_t wv[4] = {xa[gi].x, xa[gi].y, xa[gi].z, xa[gi].w};
        float x[8], v[8], rq[8], dq[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[2 * i] = __uint_as_float(wv[i] << 16);
          x[2 * i + 1] = __uint_as_float(wv[i] & 0xffff0000u);
        }
        // Eq. 1 with the straight-through estimator, the arithmetic of quant_act(): an element is
        // clipped iff |rne(x/s) + Z - mid| > half
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
        *reinterpret_cast<uint4*>(stg64(ob, lane, gi)) =
            make_uint4(pk2b(v[0], v[1]), pk2b(v[2], v[3]), pk2b(v[4], v[5]), pk2b(v[6], v[7]));
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        if (static_cast<int64_t>(t) * SB_ROWS + q * 32 < a.M) tma_store_2d(&tmDX, ob, half * 32, t * SB_ROWS + q * 32);
        tma_store_commit();
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) xa[i] = xb[i];
    }
    if (!ok && lane == 0) {
      record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
      *abort_flag = 1;
    }
    // per-warp partial sums of dS_x and dZ_x (summed in fixed order by the finalize launch)
    acc_s = warp_sum(acc_s);
    acc_c = warp_sum(acc_c);
    if (lane == 0) {
      float* pp = a.dxpart + (static_cast<int64_t>(blockIdx.x) * SB_WORKERS + e) * 2;
      pp[0] = acc_s;
      pp[1] = -xq.s * acc_c;
    }
    // ---- the CTA's weight-gradient partial: rows of the unfrozen channels only, and the column sums
    if (ok && half < a.nh) {
      bool g = *abort_flag ? false : mbar_wait(&ctl->d2_full, 0);
      if (__all_sync(0xffffffffu, g)) {
        tc_fence_after();
        const int nch = half * 128 + row;                   // channel of this lane's TMEM row
        int rank = nch;
        if (a.k_sel < a.N) {
          int lo = 0, hi = a.k_sel;                         // lower bound of nch in idx
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(a.idx + mid) < nch) lo = mid + 1; else hi = mid;
          }
          rank = (lo < a.k_sel && __ldg(a.idx + lo) == nch) ? lo : -1;
        }
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + D2_COL0 + half * D2_STRIDE;
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t r[32];
          tmem_ld_32x32(t_row + c0, r);
          tmem_wait_ld();
          if (rank >= 0) {
            float4* dst = reinterpret_cast<float4*>(a.P + (static_cast<int64_t>(blockIdx.x) * a.k_sel + rank) * 64 + c0);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]), __uint_as_float(r[4 * i + 2]),
                                   __uint_as_float(r[4 * i + 3]));
          }
        }
        uint32_t r1[32];
        tmem_ld_32x16(t_row + 64, r1);
        tmem_wait_ld();
        if (a.colsum) a.colsum[static_cast<int64_t>(blockIdx.x) * a.N + nch] = __uint_as_float(r1[0]);
      } else if (lane == 0) {
        record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
      }
    }
    if (lane == 0) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace

bool skinny_bwd_applies(int64_t M, int64_t N, int64_t K, int act_bf16) {
  return act_bf16 && M >= 1 && K == 64 && (N == 128 || N == 256);
}

int skinny_bwd_grid(int64_t M, int sm_count) {
  const int64_t tiles = ceil_div(M, SB_ROWS);
  return static_cast<int>(tiles < sm_count ? tiles : sm_count);
}

int run_skinny_bwd(int64_t M, int64_t N, const void* dY, const void* X, void* dX, const float* W, const bf16* what,
                   const float* s_w, int w_bits, const float* s_x, const float* z_x, int x_bits, int x_sym,
                   const int32_t* idx, int64_t k_sel, float* P, float* colsum, float* dxpart, int* status,
                   int sm_count, cudaStream_t st) {
  if (!skinny_bwd_applies(M, N, 64, 1)) return EFQAT_ERR_SHAPE;
  SkinnyBwdArgs a = {};
  a.M = M; a.N = static_cast<int>(N); a.nh = a.N / 128;
  a.tiles = static_cast<int>(ceil_div(M, SB_ROWS));
  a.W = W; a.what = what; a.s_w = s_w; a.w_bits = w_bits;
  a.s_x = s_x; a.z_x = z_x; a.x_bits = x_bits; a.x_sym = x_sym;
  a.idx = idx; a.k_sel = static_cast<int>(k_sel);
  a.P = P; a.colsum = colsum; a.dxpart = dxpart; a.status = status;
  CUtensorMap tmDY, tmX, tmDX;
  if (tensor_map_2d(&tmDY, dY, 1, M, N, N, SB_ROWS, 128) != EFQAT_OK) return EFQAT_ERR_CUDA;
  if (tensor_map_2d(&tmX, X, 1, M, 64, 64, SB_ROWS, 128) != EFQAT_OK) return EFQAT_ERR_CUDA;
  if (tensor_map_2d(&tmDX, dX, 1, M, 64, 64, 32, 64) != EFQAT_OK) return EFQAT_ERR_CUDA;
  const size_t smem = static_cast<size_t>(a.N) * 128 + 4 * T16K + SB_STAGES * HALF_BYTES + SB_WORKERS * 2 * 2048 +
                      sizeof(SbCtl);
  if (cudaFuncSetAttribute(skinny_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
      cudaSuccess)
    return EFQAT_ERR_CUDA;
  count_launches(1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(skinny_bwd_grid(M, sm_count)));
  cfg.blockDim = dim3(SB_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, skinny_bwd_kernel, tmDY, tmX, tmDX, a) != cudaSuccess) return EFQAT_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
}

}  // namespace efqat
