// bf16 x bf16 -> fp32 GEMM core on the 5th-generation tensor cores (tcgen05 / TMEM),
// operands staged by TMA into 128-byte-swizzled shared memory, with three fused epilogues:
//   EPI_FWD : Y = s_x * s_w[n] * acc + bias[n]                         (forward, Section 3.1)
//   EPI_DX  : dX = acc * [x not clipped]; partial sums of dS_x, dZ_x   (Eq. 5 + STE)
//   EPI_PART: fp32 partial products of the (partial) weight gradient   (Algorithm 1)
//
// One CTA computes one 128 x BN output tile (optionally one split of the contraction):
//   warp 0  lane 0 : TMA producer over a ring of shared-memory stages
//   warp 1  lane 0 : issues tcgen05.mma; warp 1 also owns the TMEM allocation
//   warps 2..5     : epilogue, each reading its 32-lane quarter of the accumulator
// Either operand may be stored with the contraction dimension contiguous ("K-major") or
// with the other dimension contiguous ("MN-major"); the shared-memory and instruction
// descriptors carry the difference, so no transposed copies are ever made.
#include <stdio.h>

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
static const int GEMM_THREADS = 192;

struct GemmParams {
  int64_t Mr, Nc;
  int nkb;            // number of BK blocks along the contraction
  int BN;             // tile columns (multiple of 16, <= 256)
  int stages;
  int b_stage_bytes;
  int tmem_cols;
  int splits;
  int out_bf16;
  void* out;
  int64_t ldo;
  const float* col_scale;
  const float* col_bias;
  const ActQ* xq;
  const void* X;
  int x_dtype;
  float* partials;
  int64_t split_stride;
  int64_t part_cols;
  int* status;
};

struct __align__(8) SmemCtl {
  uint64_t full[MAX_STAGES];
  uint64_t empty[MAX_STAGES];
  uint64_t acc_full;
  uint32_t tmem_base;
  int abort_flag;
  float red[4][2];
};

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Stores 8 consecutive outputs of one row (16-byte aligned by the N % 8 / K % 8 contract).
__device__ __forceinline__ void store8(void* base, int64_t elem_off, const float* v, int as_bf16) {
  if (as_bf16) {
    uint4 o;
    o.x = pack2(v[0], v[1]); o.y = pack2(v[2], v[3]); o.z = pack2(v[4], v[5]); o.w = pack2(v[6], v[7]);
    *reinterpret_cast<uint4*>(static_cast<bf16*>(base) + elem_off) = o;
  } else {
    float4* p = reinterpret_cast<float4*>(static_cast<float*>(base) + elem_off);
    p[0] = make_float4(v[0], v[1], v[2], v[3]);
    p[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}
__device__ __forceinline__ void load8(const void* base, int64_t elem_off, float* v, int is_bf16) {
  if (is_bf16) {
    const uint4 r = __ldg(reinterpret_cast<const uint4*>(static_cast<const bf16*>(base) + elem_off));
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  } else {
    const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem_off);
    const float4 a = __ldg(p), b = __ldg(p + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <int A_MN, int B_MN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle atoms of TMA and UMMA
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int stage_bytes = A_STAGE_BYTES + p.b_stage_bytes;
  SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + p.stages * stage_bytes);
  float* s_scale = reinterpret_cast<float*>(ctl + 1);   // [BN] (EPI_FWD)
  float* s_bias = s_scale + 256;                         // [BN]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * p.BN;
  const int m0 = blockIdx.y * BM;
  const int split = blockIdx.z;
  const int kb_begin = static_cast<int>(static_cast<int64_t>(split) * p.nkb / p.splits);
  const int kb_end = static_cast<int>(static_cast<int64_t>(split + 1) * p.nkb / p.splits);
  // columns of this tile that exist, rounded up to the UMMA N granularity
  int n_eff = static_cast<int>(p.Nc - n0);
  if (n_eff > p.BN) n_eff = p.BN;
  n_eff = (n_eff + 15) & ~15;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    mbar_init(&ctl->acc_full, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, static_cast<uint32_t>(p.tmem_cols));
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      const int b_chunks = (n_eff + 63) >> 6;
      const uint32_t tx = A_STAGE_BYTES + (B_MN ? b_chunks * CHUNK_BYTES : p.BN * BK * 2);
      int it = 0;
      for (int kb = kb_begin; kb < kb_end && !*abort_flag; ++kb, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&ctl->empty[s], ph ^ 1)) {
          record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
          *abort_flag = 1;
          break;
        }
        uint8_t* sa = smem + s * stage_bytes;
        uint8_t* sb = sa + A_STAGE_BYTES;
        mbar_arrive_expect_tx(&ctl->full[s], tx);
        if (A_MN) {
          tma_load_2d(sa, &tmA, &ctl->full[s], m0, kb * BK);
          tma_load_2d(sa + CHUNK_BYTES, &tmA, &ctl->full[s], m0 + 64, kb * BK);
        } else {
          tma_load_2d(sa, &tmA, &ctl->full[s], kb * BK, m0);
        }
        if (B_MN) {
          for (int c = 0; c < b_chunks; ++c)
            tma_load_2d(sb + c * CHUNK_BYTES, &tmB, &ctl->full[s], n0 + 64 * c, kb * BK);
        } else {
          tma_load_2d(sb, &tmB, &ctl->full[s], kb * BK, n0);
        }
      }
      // Make sure none of this CTA's bulk copies is still in flight when it exits (only
      // relevant after an abort: otherwise the MMA warp has consumed every stage).
      const int issued = it;
      for (int j = (issued > p.stages ? issued - p.stages : 0); j < issued; ++j)
        mbar_wait(&ctl->full[j % p.stages], (j / p.stages) & 1, 20000000ull);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(BM, n_eff, A_MN, B_MN);
      int it = 0;
      bool ok = true;
      for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (*abort_flag || !mbar_wait(&ctl->full[s], ph)) {
          record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
          *abort_flag = 1;
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + s * stage_bytes);
        const uint32_t b_addr = a_addr + A_STAGE_BYTES;
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          // K-major: 16 contraction elements = 32 bytes inside the swizzled 128-byte row.
          // MN-major: 16 contraction elements = 16 rows of 128 bytes = two 8-row groups.
          const uint64_t adesc = A_MN ? smem_desc_sw128(a_addr + k * 2048, CHUNK_BYTES, 1024)
                                      : smem_desc_sw128(a_addr + k * 32, 16, 1024);
          const uint64_t bdesc = B_MN ? smem_desc_sw128(b_addr + k * 2048, CHUNK_BYTES, 1024)
                                      : smem_desc_sw128(b_addr + k * 32, 16, 1024);
          umma_bf16(tmem_base, adesc, bdesc, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(&ctl->empty[s]);   // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(&ctl->acc_full);
    }
  } else {
    // ------------------------------------------------------------- epilogue (warps 2..5)
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    const int row_in_tile = q * 32 + lane;
    const int64_t row = static_cast<int64_t>(m0) + row_in_tile;
    const int et = threadIdx.x - 64;         // 0..127
    if (EPI == EPI_FWD) {
      for (int j = et; j < p.BN; j += 128) {
        const int64_t c = static_cast<int64_t>(n0) + j;
        s_scale[j] = (c < p.Nc) ? p.col_scale[c] : 0.f;
        s_bias[j] = (c < p.Nc && p.col_bias) ? p.col_bias[c] : 0.f;
      }
      epi_bar_sync();
    }
    ActQ xq;
    if (EPI != EPI_PART) xq = *p.xq;
    float acc_s = 0.f, acc_z = 0.f;
    bool ok = mbar_wait(&ctl->acc_full, 0);
    if (!ok) {
      record_status(p.status, EFQAT_DEV_WAIT_TIMEOUT);
      *abort_flag = 1;
    }
    // all lanes of a warp see the same outcome of the wait, so the branch is warp-uniform
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      for (int c0 = 0; c0 < n_eff; c0 += 32) {
        uint32_t r[32];
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c0);
        const int ncols = (n_eff - c0 >= 32) ? 32 : 16;
        if (ncols == 32) tmem_ld_32x32(taddr, r); else tmem_ld_32x16(taddr, r);
        tmem_wait_ld();
        if (EPI == EPI_PART) {
          if (row < p.Mr) {
            float* outp = static_cast<float*>(p.out) + split * p.split_stride + row;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int64_t col = static_cast<int64_t>(n0) + c0 + j;
              if (j < ncols && col < p.part_cols) outp[col * p.ldo] = __uint_as_float(r[j]);
            }
          }
        } else if (row < p.Mr) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int64_t col = static_cast<int64_t>(n0) + c0 + g * 8;
            if (g * 8 < ncols && col < p.Nc) {
              float v[8];
              if (EPI == EPI_FWD) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  v[j] = fmaf(__uint_as_float(r[g * 8 + j]) * xq.s, s_scale[c0 + g * 8 + j],
                              s_bias[c0 + g * 8 + j]);
              } else {
                float x[8];
                load8(p.X, row * p.ldo + col, x, p.x_dtype == EFQAT_BF16);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const float gx = __uint_as_float(r[g * 8 + j]);
                  const QElem e = quant_act(x[j], xq);
                  v[j] = e.flag ? 0.f : gx;
                  acc_s = fmaf(gx, e.t, acc_s);
                  acc_z += e.flag ? -gx * xq.s : 0.f;
                }
              }
              store8(p.out, row * p.ldo + col, v, p.out_bf16);
            }
          }
        }
      }
    }
    if (EPI == EPI_DX) {
      acc_s = warp_sum(acc_s);
      acc_z = warp_sum(acc_z);
      if (lane == 0) {
        ctl->red[q][0] = acc_s;
        ctl->red[q][1] = acc_z;
      }
      epi_bar_sync();
      if (et == 0) {
        const int64_t tile = static_cast<int64_t>(blockIdx.y) * gridDim.x + blockIdx.x;
        p.partials[2 * tile] = (ctl->red[0][0] + ctl->red[1][0]) + (ctl->red[2][0] + ctl->red[3][0]);
        p.partials[2 * tile + 1] = (ctl->red[0][1] + ctl->red[1][1]) + (ctl->red[2][1] + ctl->red[3][1]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

int gemm_init() {
  if (g_encode) return EFQAT_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return EFQAT_ERR_CUDA;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return EFQAT_OK;
}

// 2-D bf16 row-major matrix [rows, cols] with pitch ld (elements); box = 64 columns x box_rows rows.
static int make_map(CUtensorMap* m, const bf16* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t es[2] = {1u, 1u};
  const CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(base), dims, strides, box,
                              es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? EFQAT_OK : EFQAT_ERR_CUDA;
}

static int choose_bn(int64_t Mr, int64_t Nc, int splits, int sm_count) {
  if (Nc <= 64) return static_cast<int>(round_up(Nc, 16));
  const int64_t mt = ceil_div(Mr, BM);
  int best = 64;
  double best_cost = 1e300;
  for (int bn = 256; bn >= 64; bn -= 32) {
    const int64_t tiles = mt * ceil_div(Nc, bn) * splits;
    const double cost = static_cast<double>(ceil_div(tiles, sm_count)) * (bn + 24);
    if (cost < best_cost) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

int gemm_dx_num_partials(int64_t Mr, int64_t Nc) {
  // upper bound over every tile width the heuristic may pick
  return static_cast<int>(ceil_div(Mr, BM) * ceil_div(Nc, 64));
}

int gemm_choose_splits(int64_t Mr, int64_t Nc, int64_t Kc, int sm_count) {
  const int64_t nkb = ceil_div(Kc, BK);
  const int bn = (Nc <= 64) ? static_cast<int>(round_up(Nc, 16)) : (Nc <= 128 ? 128 : 256);
  const int64_t tiles = ceil_div(Mr, BM) * ceil_div(Nc, bn);
  int64_t s = ceil_div(sm_count, tiles);
  const int64_t max_s = nkb / 4 > 0 ? nkb / 4 : 1;   // at least four contraction blocks per split
  if (s > max_s) s = max_s;
  if (s > 64) s = 64;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}

template <int A_MN, int B_MN, int EPI>
static int launch(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, dim3 grid, size_t smem,
                  cudaStream_t st) {
  auto kern = gemm_kernel<A_MN, B_MN, EPI>;
  static bool configured[64] = {};   // per instantiation and device
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return EFQAT_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return EFQAT_ERR_CUDA;
    configured[dev] = true;
  }
  count_launches(1);
  kern<<<grid, GEMM_THREADS, smem, st>>>(ta, tb, p);
  return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
}

int run_gemm(const GemmArgs& a, int sm_count, cudaStream_t st, int* tiles_out) {
  if (a.Mr < 1 || a.Nc < 1 || a.Kc < 1) return EFQAT_ERR_SHAPE;
  int rc = gemm_init();
  if (rc != EFQAT_OK) return rc;
  GemmParams p = {};
  p.Mr = a.Mr;
  p.Nc = a.Nc;
  p.nkb = static_cast<int>(ceil_div(a.Kc, BK));
  p.splits = (a.epi == EPI_PART) ? a.splits : 1;
  if (p.splits < 1 || p.splits > p.nkb) return EFQAT_ERR_SHAPE;
  if (a.epi == EPI_PART) {
    p.BN = (a.Nc <= 64) ? static_cast<int>(round_up(a.Nc, 16)) : (a.Nc <= 128 ? 128 : 256);
  } else {
    p.BN = choose_bn(a.Mr, a.Nc, 1, sm_count);
  }
  p.b_stage_bytes = static_cast<int>(a.b_mn ? ceil_div(p.BN, 64) * CHUNK_BYTES : p.BN * BK * 2);
  p.b_stage_bytes = static_cast<int>(round_up(p.b_stage_bytes, 1024));
  const int stage_bytes = A_STAGE_BYTES + p.b_stage_bytes;
  const int ctl_bytes = static_cast<int>(sizeof(SmemCtl)) + 2 * 256 * 4;
  int stages = (227 * 1024 - 1024 - ctl_bytes) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return EFQAT_ERR_SHAPE;
  p.stages = stages;
  int cols = 32;
  while (cols < p.BN) cols <<= 1;
  p.tmem_cols = cols;
  p.out_bf16 = a.out_bf16;
  p.out = a.out;
  p.ldo = a.ldo;
  p.col_scale = a.col_scale;
  p.col_bias = a.col_bias;
  p.xq = a.xq;
  p.X = a.X;
  p.x_dtype = a.x_dtype;
  p.partials = a.partials;
  p.split_stride = a.split_stride;
  p.part_cols = a.part_cols;
  p.status = a.status;

  CUtensorMap ta, tb;
  rc = a.a_mn ? make_map(&ta, a.A, a.Kc, a.Mr, a.lda, BK) : make_map(&ta, a.A, a.Mr, a.Kc, a.lda, BM);
  if (rc != EFQAT_OK) return rc;
  rc = a.b_mn ? make_map(&tb, a.B, a.Kc, a.Nc, a.ldb, BK) : make_map(&tb, a.B, a.Nc, a.Kc, a.ldb, p.BN);
  if (rc != EFQAT_OK) return rc;

  const dim3 grid(static_cast<unsigned>(ceil_div(a.Nc, p.BN)), static_cast<unsigned>(ceil_div(a.Mr, BM)),
                  static_cast<unsigned>(p.splits));
  const size_t smem = static_cast<size_t>(stages) * stage_bytes + ctl_bytes + 1024;
  if (tiles_out) *tiles_out = static_cast<int>(grid.x * grid.y);

#define EFQAT_LAUNCH(AM, BMj, E) return launch<AM, BMj, E>(ta, tb, p, grid, smem, st)
  if (a.epi == EPI_FWD && !a.a_mn && !a.b_mn) EFQAT_LAUNCH(0, 0, EPI_FWD);
  if (a.epi == EPI_DX && !a.a_mn && a.b_mn) EFQAT_LAUNCH(0, 1, EPI_DX);
  if (a.epi == EPI_PART && a.a_mn && a.b_mn) EFQAT_LAUNCH(1, 1, EPI_PART);
  if (a.epi == EPI_PART && !a.a_mn && !a.b_mn) EFQAT_LAUNCH(0, 0, EPI_PART);
  if (a.epi == EPI_PART && !a.a_mn && a.b_mn) EFQAT_LAUNCH(0, 1, EPI_PART);
  if (a.epi == EPI_PART && a.a_mn && !a.b_mn) EFQAT_LAUNCH(1, 0, EPI_PART);
#undef EFQAT_LAUNCH
  return EFQAT_ERR_UNIMPL;
}

}  // namespace efqat
