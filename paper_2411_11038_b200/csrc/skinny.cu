// Forward of layers with a short contraction (K = 64: the 1x1 convolutions of the first ResNet
// stage) in ONE launch that touches each tensor once.  Such a layer moves 2 bytes of X
// and 2 N / K bytes of Y per 2 N flop per element of X: far below the machine's flop-per-byte
// ridge, so HBM traffic and the latency chain per tile decide its time, not the tensor pipe.
// The general path (quantizer launch writing a code matrix, then a GEMM launch reading it back,
// one persistent CTA per SM) pays a second pass over X and has ten warps per SM to hide the
// TMEM-load / store latencies of a tile whose main loop is a single k-block.  Here:
//   * fake-quant is the operand producer (Eq. 1): every thread loads 16 bytes of raw X with a
//     coalesced global load, quantizes in registers and writes the centred integer codes into
//     the 128-byte-swizzled shared-memory tile that tcgen05.mma reads; no code matrix exists;
//   * the layer's weight codes (Eq. 3) are quantized once per CTA into shared memory and stay;
//   * the accumulator lives in TMEM; the epilogue (scale, bias, cast) stages 32 rows x 128 bytes
//     per warp in swizzled shared memory and hands them to the TMA unit, so global memory sees
//     whole 128-byte row segments (a lane owns a row: direct stores would put 32 half-filled
//     sectors into every request and the load/store unit becomes the bound);
//   * CTAs are small (256 threads, <= 256 TMEM columns), so two to four of them share an SM
//     and overlap one another's load, MMA and store phases.
#include "internal.h"
#include "ptx.cuh"

namespace efqat {

using namespace ptx;

namespace {

const int SK_THREADS = 256;
const int SK_ROWS = 128;            // rows of X per tile = UMMA M = TMEM lanes

struct SkinnyFwdArgs {
  int64_t M, N;
  int K;                            // 64 or 128
  int BN;                           // output columns per CTA (multiple of 64, <= 256)
  int tmem_cols;                    // power of two >= BN
  int tiles;                        // ceil(M / 128)
  const void* X; void* Y;
  const float* W; const bf16* codes16;      // weights: fp32 to quantize here, or cached bf16 codes
  const float* s_w; const float* s_x; const float* z_x; const float* bias;
  int w_bits, x_bits, x_sym;
  int* status;
  int stages, stg_bufs;             // persistent form: X tiles in flight, staging buffers per epilogue warp
};

// 16-byte piece j (0..7) of row r inside a [rows x 64 bf16] tile in the canonical K-major
// 128-byte-swizzle layout (8-row groups of 1024 bytes).
__device__ __forceinline__ uint32_t sw128_off(int r, int j) { return r * 128 + ((j ^ (r & 7)) << 4); }

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ uint32_t pk(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <typename T, int KB /* k-blocks of 64: 1 or 2 */>
__global__ void __launch_bounds__(SK_THREADS, 2) skinny_fwd_kernel(const __grid_constant__ CUtensorMap tmY,
                                                                const SkinnyFwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];         // swizzle atoms need 1024-byte alignment
  uint8_t* a_tile = smem;                                   // [KB][128 rows][128 B]
  uint8_t* b_tile = a_tile + KB * SK_ROWS * 128;            // [KB][BN rows][128 B]
  uint8_t* stage = b_tile + KB * a.BN * 128;                // [8 warps][2 buffers][32 rows][128 B] output staging
  __shared__ __align__(8) uint64_t mma_bar;
  __shared__ uint32_t tmem_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.y * a.BN;
  int bn = static_cast<int>(a.N - n0);
  if (bn > a.BN) bn = a.BN;                                 // live columns of this CTA (multiple of 64)

  if (tid == 0) {
    mbar_init(&mma_bar, 1);
    fence_barrier_init();
    prefetch_tmap(&tmY);
  }
  if (warp == 0) {
    tmem_alloc(&tmem_slot, a.tmem_cols);
    tmem_relinquish();
  }
  pdl_trigger();
  pdl_wait();

  // ---- weights of this CTA's columns -> codes in the B tile (once)
  bool bad_scale = false;
  for (int p = tid; p < a.BN * KB * 8; p += SK_THREADS) {
    const int n = p / (KB * 8), jj = p - n * (KB * 8);
    const int kb = jj >> 3, j = jj & 7;
    uint4 o = make_uint4(0u, 0u, 0u, 0u);
    if (n < bn) {
      const int64_t g = static_cast<int64_t>(n0 + n) * a.K + jj * 8;
      if (a.codes16) {
        o = __ldg(reinterpret_cast<const uint4*>(a.codes16 + g));
      } else {
        float sw = __ldg(a.s_w + n0 + n);
        if (!scale_ok(sw)) {
          bad_scale = true;
          sw = 1.f;
        }
        const RowQ rq = make_rowq(sw, a.w_bits);
        float v[8];
        load8<float>(a.W + g, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = quant_weight(v[i], rq).c0;
        o = make_uint4(pk(v[0], v[1]), pk(v[2], v[3]), pk(v[4], v[5]), pk(v[6], v[7]));
      }
    }
    *reinterpret_cast<uint4*>(b_tile + kb * a.BN * 128 + sw128_off(n, j)) = o;
  }
  bool bad_x;
  const ActQ xq = make_actq(a.s_x, a.z_x, a.x_bits, a.x_sym, &bad_x);
  if ((bad_scale || (bad_x && tid == 0)) && blockIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const uint32_t idesc = instr_desc_bf16(SK_ROWS, bn, 0, 0);
  const T* X = static_cast<const T*>(a.X);
  constexpr int PIECES = SK_ROWS * KB * 8 / SK_THREADS;     // 16-byte pieces of the A tile per thread: 4 or 8

  // raw X of a tile, one 8-element piece per (thread, i), kept as loaded (16 bytes of bf16 or 32
  // of fp32) until the producer step: coalesced, every sector read whole
  constexpr int RAW = sizeof(T) == 2 ? 1 : 2;               // uint4 registers per piece
  uint4 xraw[PIECES][RAW];
  auto load_tile = [&](int t) {
#pragma unroll
    for (int i = 0; i < PIECES; ++i) {
      const int p = tid + i * SK_THREADS;
      const int r = p / (KB * 8), jj = p - r * (KB * 8);
      const int64_t m = static_cast<int64_t>(t) * SK_ROWS + r;
#pragma unroll
      for (int u = 0; u < RAW; ++u)
        xraw[i][u] = (m < a.M) ? __ldg(reinterpret_cast<const uint4*>(X + m * a.K + jj * 8) + u) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  auto unpack = [&](const uint4 (&raw)[RAW], float (&v)[8]) {
    if (sizeof(T) == 2) {
      const uint32_t w[4] = {raw[0].x, raw[0].y, raw[0].z, raw[0].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
    } else {
      const uint4 lo = raw[0], hi = raw[RAW - 1];
      v[0] = __uint_as_float(lo.x); v[1] = __uint_as_float(lo.y); v[2] = __uint_as_float(lo.z); v[3] = __uint_as_float(lo.w);
      v[4] = __uint_as_float(hi.x); v[5] = __uint_as_float(hi.y); v[6] = __uint_as_float(hi.z); v[7] = __uint_as_float(hi.w);
    }
  };

  const float c_lo = xq.lo - xq.zr, c_hi = xq.hi - xq.zr;
  int t = blockIdx.x;
  if (t < a.tiles) load_tile(t);
  uint32_t phase = 0;
  int st_it = 0;                    // staging rounds so far (this warp): selects the buffer
  bool ok = true;
  for (; t < a.tiles && ok; t += gridDim.x) {
    // ---- operand producer: Eq. 1 in registers, centred codes into the swizzled A tile
#pragma unroll
    for (int i = 0; i < PIECES; ++i) {
      const int p = tid + i * SK_THREADS;
      const int r = p / (KB * 8), jj = p - r * (KB * 8);
      float c[8];
      unpack(xraw[i], c);            // rows past M were loaded as zeros, whose centred code is 0
      // centred code of Eq. 1: clamp(rne(x / s) + Zr, lo, hi) - Zr = clamp(rne(x / s), lo - Zr, hi - Zr),
      // all operands integers far below 2^23, so both forms are exact and equal
#pragma unroll
      for (int e = 0; e < 8; ++e) c[e] = fminf(fmaxf(rne_small(__fmul_rn(c[e], xq.rinv)), c_lo), c_hi);
      *reinterpret_cast<uint4*>(a_tile + (jj >> 3) * SK_ROWS * 128 + sw128_off(r, jj & 7)) =
          make_uint4(pk(c[0], c[1]), pk(c[2], c[3]), pk(c[4], c[5]), pk(c[6], c[7]));
    }
    fence_proxy_async();            // generic-proxy writes of the tile become visible to the MMA's async proxy
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t a_addr = smem_u32(a_tile), b_addr = smem_u32(b_tile);
#pragma unroll
      for (int kb = 0; kb < KB; ++kb)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem_base, smem_desc_sw128(a_addr + kb * SK_ROWS * 128 + k * 32, 16, 1024),
                    smem_desc_sw128(b_addr + kb * a.BN * 128 + k * 32, 16, 1024), idesc, (kb | k) ? 1u : 0u);
      umma_commit(&mma_bar);
    }
    // the next tile's X travels while this tile's MMA and epilogue run
    const int tn = t + gridDim.x;
    if (tn < a.tiles) load_tile(tn);
    // one thread polls the MMA's barrier; the others park at the block barrier, which costs no
    // issue slots (the CTA sharing this SM is in its producer or epilogue phase meanwhile)
    if (tid == 0) ok = mbar_wait(&mma_bar, phase);
    phase ^= 1;
    if (!__syncthreads_and(ok)) {
      if (tid == 0) record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
      ok = false;
      break;
    }
    tc_fence_after();
    // ---- epilogue: warp w reads TMEM lane quarter w % 4, column half w / 4, 128 bytes of output
    // columns per round: registers -> swizzled staging -> one bulk tensor store (clipped at row M)
    {
      constexpr int RC = 128 / sizeof(T);                     // output columns per round: 64 (bf16) / 32 (fp32)
      const int q = warp & 3, h = warp >> 2;
      const int rounds = bn / RC;                             // bn is a multiple of 64
      const int rd0 = h ? (rounds + 1) / 2 : 0, rd1 = h ? rounds : (rounds + 1) / 2;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
      const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int rd = rd0; rd < rd1; ++rd, ++st_it) {
        const int c0 = rd * RC;
        uint8_t* stg = stage + (warp * 2 + (st_it & 1)) * 4096;
        uint32_t r[RC];
        tmem_ld_32x32(t_row + c0, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        if (RC == 64) tmem_ld_32x32(t_row + c0 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[RC - 32]));
        if (lane == 0) tma_store_wait_read1();                // the store two rounds back has read this buffer
        tmem_wait_ld();
        __syncwarp();
#pragma unroll
        for (int g = 0; g < RC / 8; ++g) {
          {
            // column scales and biases: every lane reads the same 32 bytes (one L1 line, broadcast)
            const float4 s0 = __ldg(reinterpret_cast<const float4*>(a.s_w + n0 + c0 + g * 8));
            const float4 s1 = __ldg(reinterpret_cast<const float4*>(a.s_w + n0 + c0 + g * 8) + 1);
            const float4 b0 = a.bias ? __ldg(reinterpret_cast<const float4*>(a.bias + n0 + c0 + g * 8)) : zero4;
            const float4 b1 = a.bias ? __ldg(reinterpret_cast<const float4*>(a.bias + n0 + c0 + g * 8) + 1) : zero4;
            const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            float v[8];
            // Y = s_x (s_w[n] acc) + b[n]: a lane owns a row, so any per-column preparation would be
            // per-element work here; two roundings instead of one, inside the fp32 class either way
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = fmaf(__uint_as_float(r[g * 8 + e]) * sv[e], xq.s, bv[e]);
            if (sizeof(T) == 2) {
              *reinterpret_cast<uint4*>(stg + sw128_off(lane, g)) =
                  make_uint4(pk(v[0], v[1]), pk(v[2], v[3]), pk(v[4], v[5]), pk(v[6], v[7]));
            } else {
              *reinterpret_cast<float4*>(stg + sw128_off(lane, 2 * g)) = make_float4(v[0], v[1], v[2], v[3]);
              *reinterpret_cast<float4*>(stg + sw128_off(lane, 2 * g + 1)) = make_float4(v[4], v[5], v[6], v[7]);
            }
          }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmY, stg, n0 + c0, t * SK_ROWS + q * 32);
          tma_store_commit();
        }
      }
    }
    tc_fence_before();
    __syncthreads();                // accumulator and A tile are free again
  }
  if (lane == 0) tma_store_wait_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, a.tmem_cols);
}


// ---------------------------------------------------------------------------------------------
// The same forward as a persistent, warp-specialised kernel for bf16 activations and up to 256
// output columns: one CTA per SM, warp 0 brings raw X tiles into a ring with TMA, warps 2..9 turn
// each tile into centred codes (Eq. 1) in one of two operand buffers and run the epilogue of the
// previous tile, warp 1 issues the MMAs into one of two TMEM accumulators.  Load, quantizer, MMA
// and epilogue of neighbouring tiles overlap inside the CTA, so a tile costs what its bytes cost.
const int WS_THREADS = 320;
const int WS_MAX_STAGES = 3;
const int WS_T16K = SK_ROWS * 128;

struct __align__(16) WsCtl {
  uint64_t full[WS_MAX_STAGES], empty[WS_MAX_STAGES];
  uint64_t xc_full[2], xc_empty[2];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

template <int KB /* 64-wide k-blocks of the contraction: 1 or 2 */, int NW /* worker warps: 8 or 16 */>
__global__ void __launch_bounds__(64 + 32 * NW, 1)
skinny_fwd_ws_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY,
                     const SkinnyFwdArgs a) {
  constexpr int TILE = KB * WS_T16K;                       // one X tile / one operand buffer
  constexpr int WS_STAGES = KB == 1 ? 3 : 2;               // X tiles in flight (compile time: the stage index is n % WS_STAGES)
  constexpr int STG_BUFS = (KB == 1 && NW == 8) ? 2 : 1;   // staging buffers per epilogue warp
  constexpr int G = NW / 4;                                // worker warps per TMEM lane quarter
  constexpr int THREADS = 64 + 32 * NW;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* b_tile = smem;                                  // [KB][BN rows][128 B] weight codes, K-major
  uint8_t* xc_t = b_tile + KB * a.BN * 128;                // [2][KB][128 rows][128 B] centred activation codes
  uint8_t* ring = xc_t + 2 * TILE;                         // [stages][KB][128 rows][128 B] raw X tiles
  uint8_t* stage = ring + WS_STAGES * TILE;                // [8 warps][stg_bufs][32 rows][128 B] output staging
  float* sc = reinterpret_cast<float*>(stage + NW * STG_BUFS * 4096);   // [BN] s_x * s_w[n]
  float* bi = sc + a.BN;                                   // [BN] bias[n]
  WsCtl* ctl = reinterpret_cast<WsCtl*>(bi + a.BN);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.y * a.BN;
  int bn = static_cast<int>(a.N - n0);
  if (bn > a.BN) bn = a.BN;
  if (tid == 0) {
    for (int s = 0; s < WS_STAGES; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], NW);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->xc_full[b], NW);
      mbar_init(&ctl->xc_empty[b], 1);
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], NW);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmX);
    prefetch_tmap(&tmY);
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, 512);
    tmem_relinquish();
  }
  pdl_trigger();
  pdl_wait();
  __syncthreads();
  const int my_tiles = (a.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  // the first tiles travel while the weights are quantized
  if (tid == 0) {
    for (int n = 0; n < my_tiles && n < WS_STAGES; ++n) {
      mbar_arrive_expect_tx(&ctl->full[n], TILE);
      for (int kb = 0; kb < KB; ++kb)
        tma_load_2d(ring + n * TILE + kb * WS_T16K, &tmX, &ctl->full[n], kb * 64, (blockIdx.x + n * gridDim.x) * SK_ROWS);
    }
  }
  bool bad_scale = false;
  for (int n = tid - 32; n >= 0 && n < a.BN; n += THREADS - 32) {
    if (n >= bn) {
#pragma unroll
      for (int j = 0; j < 8 * KB; ++j)
        *reinterpret_cast<uint4*>(b_tile + (j >> 3) * a.BN * 128 + sw128_off(n, j & 7)) = make_uint4(0u, 0u, 0u, 0u);
      sc[n] = 0.f;
      bi[n] = 0.f;
      continue;
    }
    float sw = __ldg(a.s_w + n0 + n);
    if (!scale_ok(sw)) {
      bad_scale = true;
      sw = 1.f;
    }
    if (a.codes16) {
      uint4 o[8 * KB];
#pragma unroll
      for (int j = 0; j < 8 * KB; ++j)
        o[j] = __ldg(reinterpret_cast<const uint4*>(a.codes16 + static_cast<int64_t>(n0 + n) * (64 * KB)) + j);
#pragma unroll
      for (int j = 0; j < 8 * KB; ++j) *reinterpret_cast<uint4*>(b_tile + (j >> 3) * a.BN * 128 + sw128_off(n, j & 7)) = o[j];
    } else {
      float4 w4[16 * KB];
#pragma unroll
      for (int j = 0; j < 16 * KB; ++j)
        w4[j] = __ldg(reinterpret_cast<const float4*>(a.W + static_cast<int64_t>(n0 + n) * (64 * KB)) + j);
      const RowQ rq = make_rowq(sw, a.w_bits);
#pragma unroll
      for (int j = 0; j < 8 * KB; ++j) {
        const float w[8] = {w4[2 * j].x, w4[2 * j].y, w4[2 * j].z, w4[2 * j].w,
                            w4[2 * j + 1].x, w4[2 * j + 1].y, w4[2 * j + 1].z, w4[2 * j + 1].w};
        float c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) c[i] = quant_weight(w[i], rq).c0;
        *reinterpret_cast<uint4*>(b_tile + (j >> 3) * a.BN * 128 + sw128_off(n, j & 7)) =
            make_uint4(pk(c[0], c[1]), pk(c[2], c[3]), pk(c[4], c[5]), pk(c[6], c[7]));
      }
    }
    sc[n] = sw;                        // s_x folded in below, once it is known
    bi[n] = a.bias ? __ldg(a.bias + n0 + n) : 0.f;
  }
  bool bad_x;
  const ActQ xq = make_actq(a.s_x, a.z_x, a.x_bits, a.x_sym, &bad_x);
  if ((bad_scale || (bad_x && tid == 0)) && blockIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
  __syncthreads();
  for (int n = tid; n < a.BN; n += THREADS) sc[n] *= xq.s;
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      bool live = true;
      int n = WS_STAGES;
      for (; n < my_tiles && live; ++n) {
        const int s = n % WS_STAGES;
        if (*abort_flag || !mbar_wait(&ctl->empty[s], ((n / WS_STAGES) & 1) ^ 1)) { live = false; break; }
        mbar_arrive_expect_tx(&ctl->full[s], TILE);
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d(ring + s * TILE + kb * WS_T16K, &tmX, &ctl->full[s], kb * 64, (blockIdx.x + n * gridDim.x) * SK_ROWS);
      }
      if (!live) {
        record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
        *abort_flag = 1;
        const int issued = n < my_tiles ? n : my_tiles;
        for (int j = (issued > WS_STAGES ? issued - WS_STAGES : 0); j < issued; ++j)
          mbar_wait(&ctl->full[j % WS_STAGES], (j / WS_STAGES) & 1, 20000000ull);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(SK_ROWS, bn, 0, 0);
      const uint32_t b_addr = smem_u32(b_tile);
      bool ok = true;
      for (int n = 0; n < my_tiles && ok; ++n) {
        const int b = n & 1;
        if (*abort_flag || !mbar_wait(&ctl->acc_empty[b], ((n >> 1) & 1) ^ 1)) { ok = false; break; }
        if (*abort_flag || !mbar_wait(&ctl->xc_full[b], (n >> 1) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(xc_t + b * TILE);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16(tmem_base + b * 256, smem_desc_sw128(a_addr + kb * WS_T16K + k * 32, 16, 1024),
                      smem_desc_sw128(b_addr + kb * a.BN * 128 + k * 32, 16, 1024), idesc, (kb | k) ? 1u : 0u);
        umma_commit(&ctl->acc_full[b]);
        umma_commit(&ctl->xc_empty[b]);
      }
      if (!ok) {
        record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
        *abort_flag = 1;
        umma_commit(&ctl->drain);
        mbar_wait(&ctl->drain, 0, 20000000ull);
      }
    }
  } else {
    const int e = warp - 2, q = warp & 3, h = e >> 2;
    const int row = q * 32 + lane;
    const float c_lo = xq.lo - xq.zr, c_hi = xq.hi - xq.zr;
    int st_it = 0;
    bool ok = true;
    // Eq. 1 on this lane's 32 * KB values (row `row`, half h of its pieces) of tile number n
    constexpr int NP = 8 * KB / G;                           // 16-byte pieces per lane
    auto piece_off = [&](int i) { const int p = h * NP + i; return (p >> 3) * WS_T16K + sw128_off(row, p & 7); };
    auto quant_tile = [&](int n) -> bool {
      const int s = n % WS_STAGES, b = n & 1;
      bool g = *abort_flag ? false : mbar_wait(&ctl->full[s], (n / WS_STAGES) & 1);
      if (!__all_sync(0xffffffffu, g)) return false;
      uint4 xr[NP];
#pragma unroll
      for (int i = 0; i < NP; ++i) xr[i] = *reinterpret_cast<const uint4*>(ring + s * TILE + piece_off(i));
      fence_proxy_async();           // the bulk copy that refills the stage is ordered behind these reads
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->empty[s]);
      g = *abort_flag ? false : mbar_wait(&ctl->xc_empty[b], ((n >> 1) & 1) ^ 1);
      if (!__all_sync(0xffffffffu, g)) return false;
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        const uint32_t wv[4] = {xr[i].x, xr[i].y, xr[i].z, xr[i].w};
        float c[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          c[2 * j] = __uint_as_float(wv[j] << 16);
          c[2 * j + 1] = __uint_as_float(wv[j] & 0xffff0000u);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = fminf(fmaxf(rne_small(__fmul_rn(c[j], xq.rinv)), c_lo), c_hi);
        *reinterpret_cast<uint4*>(xc_t + b * TILE + piece_off(i)) =
            make_uint4(pk(c[0], c[1]), pk(c[2], c[3]), pk(c[4], c[5]), pk(c[6], c[7]));
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->xc_full[b]);
      return true;
    };
    if (my_tiles > 0) ok = quant_tile(0);
    const int rounds = bn / 64;                              // 128-byte rounds of output columns
    const int rd0 = (rounds * h + G - 1) / G, rd1 = (rounds * (h + 1) + G - 1) / G;
    for (int n = 0; n < my_tiles && ok; ++n) {
      const int t = blockIdx.x + n * gridDim.x;
      const int b = n & 1;
      if (n + 1 < my_tiles) {
        ok = quant_tile(n + 1);
        if (!ok) break;
      }
      bool g = *abort_flag ? false : mbar_wait(&ctl->acc_full[b], (n >> 1) & 1);
      if (!__all_sync(0xffffffffu, g)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 256;
      for (int rd = rd0; rd < rd1; ++rd, ++st_it) {
        const int c0 = rd * 64;
        uint8_t* stg = stage + (e * STG_BUFS + (STG_BUFS == 2 ? (st_it & 1) : 0)) * 4096;
        uint32_t r[64];
        tmem_ld_32x32(t_row + c0, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
        tmem_ld_32x32(t_row + c0 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
        if (lane == 0) {
          if (STG_BUFS == 2) tma_store_wait_read1(); else tma_store_wait_read0();
        }
        tmem_wait_ld();
        if (rd + 1 == rd1) {                                  // the accumulator is in registers: hand it back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
        }
        __syncwarp();
#pragma unroll
        for (int gi = 0; gi < 8; ++gi) {
          const float4 s0 = *reinterpret_cast<const float4*>(sc + c0 + gi * 8);
          const float4 s1 = *reinterpret_cast<const float4*>(sc + c0 + gi * 8 + 4);
          const float4 b0 = *reinterpret_cast<const float4*>(bi + c0 + gi * 8);
          const float4 b1 = *reinterpret_cast<const float4*>(bi + c0 + gi * 8 + 4);
          const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
          const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
          float v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = fmaf(__uint_as_float(r[gi * 8 + j]), sv[j], bv[j]);
          *reinterpret_cast<uint4*>(stg + sw128_off(lane, gi)) =
              make_uint4(pk(v[0], v[1]), pk(v[2], v[3]), pk(v[4], v[5]), pk(v[6], v[7]));
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (static_cast<int64_t>(t) * SK_ROWS + q * 32 < a.M) tma_store_2d(&tmY, stg, n0 + c0, t * SK_ROWS + q * 32);
          tma_store_commit();
        }
      }
      if (rd0 >= rd1) {                                       // a warp without columns still returns the accumulator
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->acc_empty[b]);
      }
    }
    if (!ok && lane == 0) {
      record_status(a.status, EFQAT_DEV_WAIT_TIMEOUT);
      *abort_flag = 1;
    }
    if (lane == 0) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace

// Contractions of 64 and, for bf16 activations (the persistent form), 128.
bool skinny_fwd_applies(int64_t M, int64_t N, int64_t K, int act_bf16) {
  return M >= 1 && (K == 64 || (K == 128 && act_bf16)) && N >= 64 && (N & 63) == 0;
}

int run_skinny_fwd(int64_t M, int64_t N, int64_t K, int act_bf16, const void* X, void* Y, const float* W,
                   const bf16* codes16, const float* s_w, const float* s_x, const float* z_x, const float* bias,
                   int w_bits, int x_bits, int x_sym, int* status, int sm_count, cudaStream_t st) {
  if (M < 1 || (K != 64 && K != 128) || N < 64 || (N & 63)) return EFQAT_ERR_SHAPE;
  SkinnyFwdArgs a = {};
  a.M = M; a.N = N; a.K = static_cast<int>(K);
  // columns per CTA: the whole layer up to 256, else equal 64-multiples of at most 256
  const int chunks = static_cast<int>(ceil_div(N, 256));
  a.BN = static_cast<int>(round_up(ceil_div(N, chunks), 64));
  a.tmem_cols = a.BN <= 64 ? 64 : (a.BN <= 128 ? 128 : 256);
  a.tiles = static_cast<int>(ceil_div(M, SK_ROWS));
  a.X = X; a.Y = Y; a.W = W; a.codes16 = codes16;
  a.s_w = s_w; a.s_x = s_x; a.z_x = z_x; a.bias = bias;
  a.w_bits = w_bits; a.x_bits = x_bits; a.x_sym = x_sym;
  a.status = status;
  if (act_bf16) {
    // persistent warp-specialised form: one CTA per SM and column chunk.  K = 128 doubles the weight,
    // operand and ring tiles: two X tiles in flight and one staging buffer per warp then fill the SM.
    const int kbs = a.K / 64;
    // Worker warps: 16 where every one of them gets a 64-column round of the epilogue (256 columns;
    // measured 2.3 -> 2.05 us per tile), else 8 (narrower tiles: 16 cost 2 us per launch; K = 128 has no
    // shared memory for 16 staging blocks).
    const int nw = (kbs == 1 && a.BN >= 256) ? 16 : 8;
    a.stages = kbs == 1 ? 3 : 2;
    a.stg_bufs = (kbs == 1 && nw == 8) ? 2 : 1;
    CUtensorMap tmX, tmY;
    if (tensor_map_2d(&tmX, X, 1, M, K, K, SK_ROWS, 128) != EFQAT_OK) return EFQAT_ERR_CUDA;
    if (tensor_map_2d(&tmY, Y, 1, M, N, N, 32, 128) != EFQAT_OK) return EFQAT_ERR_CUDA;
    const size_t smem = static_cast<size_t>(kbs) * a.BN * 128 + (2 + a.stages) * kbs * WS_T16K + nw * a.stg_bufs * 4096 +
                        2 * a.BN * sizeof(float) + sizeof(WsCtl);
    auto kern = kbs == 2 ? skinny_fwd_ws_kernel<2, 8> : (nw == 16 ? skinny_fwd_ws_kernel<1, 16> : skinny_fwd_ws_kernel<1, 8>);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
      return EFQAT_ERR_CUDA;
    int ctas = sm_count / chunks;
    if (ctas < 1) ctas = 1;
    if (ctas > a.tiles) ctas = a.tiles;
    count_launches(1);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas), static_cast<unsigned>(chunks));
    cfg.blockDim = dim3(64 + 32 * nw);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmX, tmY, a) != cudaSuccess) return EFQAT_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
  }
  const int kb = a.K / 64;
  // CTAs per SM: as many as TMEM holds (512 columns); the shared-memory request is padded so that
  // no further CTA becomes resident and then waits for TMEM columns
  int resident = 512 / a.tmem_cols;
  if (resident > 2) resident = 2;               // registers: 2 x 256 threads x up to 128
  size_t smem = static_cast<size_t>(kb) * (SK_ROWS + a.BN) * 128 + 8 * 2 * 4096;
  const int by_smem = static_cast<int>((228 * 1024) / (smem + 1024));
  if (by_smem < resident) resident = by_smem < 1 ? 1 : by_smem;
  const size_t floor_bytes = static_cast<size_t>(227 * 1024) / (resident + 1) + 1024;
  if (smem < floor_bytes) smem = floor_bytes;
  int ctas = sm_count * resident;
  if (ctas > a.tiles) ctas = a.tiles;
  auto kern = act_bf16 ? (kb == 1 ? skinny_fwd_kernel<bf16, 1> : skinny_fwd_kernel<bf16, 2>)
                       : (kb == 1 ? skinny_fwd_kernel<float, 1> : skinny_fwd_kernel<float, 2>);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
    return EFQAT_ERR_CUDA;
  count_launches(1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(ctas), static_cast<unsigned>(chunks));
  cfg.blockDim = dim3(SK_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  // Y as [M, N] with boxes of 32 rows x 128 bytes (one epilogue round of one warp)
  CUtensorMap tmY;
  if (tensor_map_2d(&tmY, Y, act_bf16 ? 1 : 0, M, N, N, 32, 128) != EFQAT_OK) return EFQAT_ERR_CUDA;
  if (cudaLaunchKernelEx(&cfg, kern, tmY, a) != cudaSuccess) return EFQAT_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
}

}  // namespace efqat
