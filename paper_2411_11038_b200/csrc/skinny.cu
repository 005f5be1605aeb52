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
};

// 16-byte piece j (0..7) of row r inside a [rows x 64 bf16] tile in the canonical K-major
// 128-byte-swizzle layout (8-row groups of 1024 bytes).
__device__ __forceinline__ uint32_t sw128_off(int r, int j) { return r * 128 + ((j ^ (r & 7)) << 4); }

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8<bf16>(const bf16* p, float (&v)[8]) {
  const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
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
  T* Y = static_cast<T*>(a.Y);
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

}  // namespace

// A contraction of 64: weight codes, operand tile and staging of two CTAs fit one SM.  At 128 the
// tiles double, one CTA per SM is left, and the general two-launch path measured faster
// (28 x 28 x 128 -> 512 at batch 64: 46 us against 57 us); the kernel itself handles both.
bool skinny_fwd_applies(int64_t M, int64_t N, int64_t K) {
  return M >= 1 && K == 64 && N >= 64 && (N & 63) == 0;
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
