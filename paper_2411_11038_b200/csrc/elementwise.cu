// Bandwidth-class kernels: quantizer producers, gathers, reductions, finalisation.
#include "internal.h"

namespace efqat {

// ------------------------------------------------------------------ parameter prep
__global__ void prep_act_kernel(const float* __restrict__ s_x, const float* __restrict__ z_x, int x_bits,
                                int x_sym, ActQ* __restrict__ out, int* status) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  ActQ p;
  float s = s_x[0];
  if (!scale_ok(s)) {
    record_status(status, EFQAT_DEV_BAD_SCALE);
    s = 1.f;
  }
  p.s = s;
  const double inv = 1.0 / static_cast<double>(s);
  p.rinv = static_cast<float>(inv);
  p.rinv_lo = static_cast<float>(inv - static_cast<double>(p.rinv));
  if (x_sym) {
    const float qs = static_cast<float>((1 << (x_bits - 1)) - 1);
    p.lo = -qs;
    p.hi = qs;
    p.zr = 0.f;
  } else {
    p.lo = 0.f;
    p.hi = static_cast<float>((1 << x_bits) - 1);
    p.zr = fminf(fmaxf(rintf(z_x[0]), p.lo), p.hi);
  }
  p.pad0 = p.pad1 = 0.f;
  *out = p;
}

void launch_prep_act(const float* s_x, const float* z_x, int x_bits, int x_sym, ActQ* out, int* status,
                     cudaStream_t st) {
  count_launches(1);
  prep_act_kernel<<<1, 32, 0, st>>>(s_x, z_x, x_bits, x_sym, out, status);
}

// ------------------------------------------------------------------ vector loads
template <typename T>
struct Vec8;
template <>
struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, float (&v)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};
template <>
struct Vec8<bf16> {
  static __device__ __forceinline__ void load(const bf16* p, float (&v)[8]) {
    const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void store8_bf16(bf16* p, const float (&v)[8]) {
  uint4 o;
  o.x = pack_bf16x2(v[0], v[1]);
  o.y = pack_bf16x2(v[2], v[3]);
  o.z = pack_bf16x2(v[4], v[5]);
  o.w = pack_bf16x2(v[6], v[7]);
  *reinterpret_cast<uint4*>(p) = o;
}

static int grid_for(int64_t work_items, int threads, int max_blocks = 148 * 16) {
  int64_t b = ceil_div(work_items, threads);
  if (b < 1) b = 1;
  if (b > max_blocks) b = max_blocks;
  return static_cast<int>(b);
}

// ------------------------------------------------------------------ activation quantizer
// out[i] = bf16(q - Zr): an exact small integer, the operand of the forward and
// weight-gradient contractions.
template <typename T>
__global__ void __launch_bounds__(256) quant_act_operand_kernel(const T* __restrict__ X, int64_t n8,
                                                                const ActQ* __restrict__ qp,
                                                                bf16* __restrict__ out) {
  const ActQ p = *qp;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n8;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[8];
    Vec8<T>::load(X + i * 8, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = quant_act(v[j], p).c0;
    store8_bf16(out + i * 8, v);
  }
}

void launch_quant_act_operand(const void* X, int dtype, int64_t count, const ActQ* q, bf16* out,
                              cudaStream_t st) {
  const int64_t n8 = count / 8;
  if (n8 == 0) return;
  const int g = grid_for(n8, 256);
  count_launches(1);
  if (dtype == EFQAT_BF16)
    quant_act_operand_kernel<bf16><<<g, 256, 0, st>>>(static_cast<const bf16*>(X), n8, q, out);
  else
    quant_act_operand_kernel<float><<<g, 256, 0, st>>>(static_cast<const float*>(X), n8, q, out);
}

template <typename T>
__global__ void quant_act_export_kernel(const T* __restrict__ X, int64_t count, const ActQ* __restrict__ qp,
                                        int32_t* __restrict__ codes, uint8_t* __restrict__ clip) {
  const ActQ p = *qp;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < count;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const QElem e = quant_act(static_cast<float>(X[i]), p);
    if (codes) codes[i] = e.code;
    if (clip) clip[i] = static_cast<uint8_t>(e.flag);
  }
}

void launch_quant_act_export(const void* X, int dtype, int64_t count, const ActQ* q, int32_t* codes,
                             uint8_t* clip, cudaStream_t st) {
  if (count == 0) return;
  const int g = grid_for(count, 256);
  count_launches(1);
  if (dtype == EFQAT_BF16)
    quant_act_export_kernel<bf16><<<g, 256, 0, st>>>(static_cast<const bf16*>(X), count, q, codes, clip);
  else
    quant_act_export_kernel<float><<<g, 256, 0, st>>>(static_cast<const float*>(X), count, q, codes, clip);
}

// ------------------------------------------------------------------ weight quantizer
// One block per output channel (row): the row's reciprocal scale is formed once.
template <int MODE>
__global__ void __launch_bounds__(256) quant_weight_operand_kernel(const float* __restrict__ W, int64_t K,
                                                                   const float* __restrict__ s_w, int w_bits,
                                                                   bf16* __restrict__ out, int* status) {
  const int64_t n = blockIdx.x;
  float s = s_w[n];
  if (!scale_ok(s)) {
    if (threadIdx.x == 0) record_status(status, EFQAT_DEV_BAD_SCALE);
    s = 1.f;
  }
  const RowQ p = make_rowq(s, w_bits);
  const float* row = W + n * K;
  bf16* orow = out + n * K;
  for (int64_t k = threadIdx.x * 4; k < K; k += blockDim.x * 4) {
    const float4 w = __ldg(reinterpret_cast<const float4*>(row + k));
    float v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float q = quant_weight(v[j], p).c0;
      v[j] = (MODE == 0) ? q : __fmul_rn(p.s, q);
    }
    uint2 o;
    o.x = pack_bf16x2(v[0], v[1]);
    o.y = pack_bf16x2(v[2], v[3]);
    *reinterpret_cast<uint2*>(orow + k) = o;
  }
}

void launch_quant_weight_operand(const float* W, int64_t N, int64_t K, const float* s_w, int w_bits, int mode,
                                 bf16* out, int* status, cudaStream_t st) {
  if (N == 0) return;
  count_launches(1);
  if (mode == 0)
    quant_weight_operand_kernel<0><<<static_cast<unsigned>(N), 256, 0, st>>>(W, K, s_w, w_bits, out, status);
  else
    quant_weight_operand_kernel<1><<<static_cast<unsigned>(N), 256, 0, st>>>(W, K, s_w, w_bits, out, status);
}

__global__ void quant_weight_export_kernel(const float* __restrict__ W, int64_t K, const float* __restrict__ s_w,
                                           int w_bits, int32_t* __restrict__ codes, uint8_t* __restrict__ clip,
                                           int* status) {
  const int64_t n = blockIdx.x;
  float s = s_w[n];
  if (!scale_ok(s)) {
    if (threadIdx.x == 0) record_status(status, EFQAT_DEV_BAD_SCALE);
    s = 1.f;
  }
  const RowQ p = make_rowq(s, w_bits);
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
    const QElem e = quant_weight(W[n * K + k], p);
    if (codes) codes[n * K + k] = e.code;
    if (clip) clip[n * K + k] = static_cast<uint8_t>(e.flag);
  }
}

void launch_quant_weight_export(const float* W, int64_t N, int64_t K, const float* s_w, int w_bits,
                                int32_t* codes, uint8_t* clip, int* status, cudaStream_t st) {
  if (N == 0) return;
  count_launches(1);
  quant_weight_export_kernel<<<static_cast<unsigned>(N), 256, 0, st>>>(W, K, s_w, w_bits, codes, clip, status);
}

// ------------------------------------------------------------------ fp32 -> bf16
__global__ void __launch_bounds__(256) to_bf16_kernel(const float* __restrict__ in, int64_t n8,
                                                      bf16* __restrict__ out) {
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < n8;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[8];
    Vec8<float>::load(in + i * 8, v);
    store8_bf16(out + i * 8, v);
  }
}
void launch_to_bf16(const float* in, int64_t count, bf16* out, cudaStream_t st) {
  const int64_t n8 = count / 8;
  if (n8 == 0) return;
  count_launches(1);
  to_bf16_kernel<<<grid_for(n8, 256), 256, 0, st>>>(in, n8, out);
}

// ------------------------------------------------------------------ gather of the selected dY columns
// out[m, j] = bf16(dY[m, idx[j]]) for j < k_sel, 0 for the pad columns up to `pitch`.
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const T* __restrict__ dY, int64_t M, int64_t N,
                                                          const int32_t* __restrict__ idx, int k_sel, int pitch,
                                                          bf16* __restrict__ out, int* status) {
  extern __shared__ int32_t s_idx[];
  for (int j = threadIdx.x; j < pitch; j += blockDim.x) {
    int32_t c = -1;
    if (j < k_sel) {
      c = idx[j];
      const bool bad = c < 0 || c >= N || (j > 0 && idx[j - 1] >= c);
      if (bad) {
        if (blockIdx.x == 0) record_status(status, EFQAT_DEV_BAD_INDEX);
        if (c < 0 || c >= N) c = -1;
      }
    }
    s_idx[j] = c;
  }
  __syncthreads();
  const int rows_per_block = 8;
  for (int64_t m0 = static_cast<int64_t>(blockIdx.x) * rows_per_block; m0 < M;
       m0 += static_cast<int64_t>(gridDim.x) * rows_per_block) {
    for (int r = 0; r < rows_per_block; ++r) {
      const int64_t m = m0 + r;
      if (m >= M) break;
      const T* src = dY + m * N;
      bf16* dst = out + m * pitch;
      for (int j = threadIdx.x; j < pitch; j += blockDim.x) {
        const int32_t c = s_idx[j];
        const float v = (c >= 0) ? static_cast<float>(src[c]) : 0.f;
        dst[j] = __float2bfloat16_rn(v);
      }
    }
  }
}

void launch_gather_cols(const void* dY, int dtype, int64_t M, int64_t N, const int32_t* idx, int64_t k_sel,
                        int64_t pitch, bf16* out, int* status, cudaStream_t st) {
  if (M == 0 || pitch == 0) return;
  const int g = grid_for(ceil_div(M, 8), 1, 148 * 8);
  const size_t sm = static_cast<size_t>(pitch) * sizeof(int32_t);
  count_launches(1);
  if (dtype == EFQAT_BF16)
    gather_cols_kernel<bf16><<<g, 256, sm, st>>>(static_cast<const bf16*>(dY), M, N, idx,
                                                 static_cast<int>(k_sel), static_cast<int>(pitch), out, status);
  else
    gather_cols_kernel<float><<<g, 256, sm, st>>>(static_cast<const float*>(dY), M, N, idx,
                                                  static_cast<int>(k_sel), static_cast<int>(pitch), out, status);
}

// ------------------------------------------------------------------ db = column sums of dY
template <typename T>
__global__ void __launch_bounds__(128) colsum_stage1_kernel(const T* __restrict__ dY, int64_t M, int64_t N,
                                                            float* __restrict__ ws) {
  const int64_t c0 = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 8;
  const int slab = blockIdx.y;
  const int64_t rows = ceil_div(M, static_cast<int64_t>(gridDim.y));
  const int64_t m_lo = slab * rows;
  const int64_t m_hi = (m_lo + rows < M) ? m_lo + rows : M;
  if (c0 >= N) return;
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  for (int64_t m = m_lo; m < m_hi; ++m) {
    float v[8];
    Vec8<T>::load(dY + m * N + c0, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] += v[j];
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) ws[static_cast<int64_t>(slab) * N + c0 + j] = acc[j];
}
__global__ void colsum_stage2_kernel(const float* __restrict__ ws, int slabs, int64_t N, float* __restrict__ db) {
  const int64_t n = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (n >= N) return;
  double acc = 0.0;
  for (int s = 0; s < slabs; ++s) acc += static_cast<double>(ws[static_cast<int64_t>(s) * N + n]);
  db[n] = static_cast<float>(acc);
}

void launch_colsum(const void* dY, int dtype, int64_t M, int64_t N, float* ws, float* db, cudaStream_t st) {
  if (N == 0) return;
  int slabs = static_cast<int>(ceil_div(M, 32));
  if (slabs > COLSUM_SLABS) slabs = COLSUM_SLABS;
  if (slabs < 1) slabs = 1;
  dim3 g(static_cast<unsigned>(ceil_div(N, 128 * 8)), slabs);
  count_launches(2);
  if (dtype == EFQAT_BF16)
    colsum_stage1_kernel<bf16><<<g, 128, 0, st>>>(static_cast<const bf16*>(dY), M, N, ws);
  else
    colsum_stage1_kernel<float><<<g, 128, 0, st>>>(static_cast<const float*>(dY), M, N, ws);
  colsum_stage2_kernel<<<static_cast<unsigned>(ceil_div(N, 256)), 256, 0, st>>>(ws, slabs, N, db);
}

// ------------------------------------------------------------------ dS_x, dZ_x: combine the per-tile partials
__global__ void __launch_bounds__(256) dx_finalize_kernel(const float* __restrict__ partials, int n,
                                                          float* __restrict__ dS_x, float* __restrict__ dZ_x) {
  __shared__ double sh[2][256];
  double a = 0.0, b = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) {
    a += static_cast<double>(partials[2 * i]);
    b += static_cast<double>(partials[2 * i + 1]);
  }
  sh[0][threadIdx.x] = a;
  sh[1][threadIdx.x] = b;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sh[0][threadIdx.x] += sh[0][threadIdx.x + o];
      sh[1][threadIdx.x] += sh[1][threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    dS_x[0] = static_cast<float>(sh[0][0]);
    dZ_x[0] = static_cast<float>(sh[1][0]);
  }
}
void launch_dx_finalize(const float* partials, int n, float* dS_x, float* dZ_x, cudaStream_t st) {
  count_launches(1);
  dx_finalize_kernel<<<1, 256, 0, st>>>(partials, n, dS_x, dZ_x);
}

// ------------------------------------------------------------------ dW: combine split partials, mask, dS_w, SGD
// One block per selected channel i (row idx[i] of W).  G = s_x * sum_splits P;
// dW_sel = G where the weight code was not clipped; dS_w = sum_k G * t_w.
__global__ void __launch_bounds__(256) dw_finalize_kernel(const float* __restrict__ P, int splits,
                                                          int64_t split_stride, int64_t K,
                                                          const float* __restrict__ W,
                                                          const float* __restrict__ s_w,
                                                          const int32_t* __restrict__ idx, int64_t N_rows,
                                                          const ActQ* __restrict__ xq, int w_bits,
                                                          float* __restrict__ dW_sel, float* __restrict__ dS_w_sel,
                                                          efqat_sgd opt, int has_opt, int* status) {
  const int64_t i = blockIdx.x;
  const int64_t n = idx ? static_cast<int64_t>(idx[i]) : i;
  if (n < 0 || n >= N_rows) {
    if (threadIdx.x == 0) record_status(status, EFQAT_DEV_BAD_INDEX);
    return;
  }
  float s = s_w[n];
  if (!scale_ok(s)) s = 1.f;   // already reported by the weight quantizer of this call
  const RowQ p = make_rowq(s, w_bits);
  const float sx = xq->s;
  const float* wrow = W + n * K;
  double acc = 0.0;
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
    float g = 0.f;
    for (int sp = 0; sp < splits; ++sp) g += P[sp * split_stride + i * K + k];
    g *= sx;
    const float w = wrow[k];
    const QElem e = quant_weight(w, p);
    const float gw = e.flag ? 0.f : g;
    dW_sel[i * K + k] = gw;
    acc += static_cast<double>(g) * static_cast<double>(e.t);
    if (has_opt) {
      const int64_t o = n * K + k;
      const float wv = opt.W_inout[o];
      const float v = opt.momentum * opt.mom_inout[o] + (gw + opt.weight_decay * wv);
      opt.mom_inout[o] = v;
      opt.W_inout[o] = wv - opt.lr * v;
    }
  }
  __shared__ double sh[8];
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += sh[w];
    dS_w_sel[i] = static_cast<float>(t);
  }
}

void launch_dw_finalize(const float* P, int splits, int64_t split_stride, int64_t k_sel, int64_t N, int64_t K,
                        const float* W, const float* s_w, const int32_t* idx_or_null, const ActQ* xq, int w_bits,
                        float* dW_sel, float* dS_w_sel, const efqat_sgd* opt, int* status, cudaStream_t st) {
  if (k_sel == 0) return;
  efqat_sgd o = {};
  if (opt) o = *opt;
  count_launches(1);
  dw_finalize_kernel<<<static_cast<unsigned>(k_sel), 256, 0, st>>>(P, splits, split_stride, K, W, s_w, idx_or_null,
                                                                  N, xq, w_bits, dW_sel, dS_w_sel, o,
                                                                  opt != nullptr, status);
}

// ------------------------------------------------------------------ MinMax initialisation (Eq. 2, Eq. 4)
template <typename T>
__global__ void __launch_bounds__(256) minmax_stage1_kernel(const T* __restrict__ x, int64_t count,
                                                            float* __restrict__ ws) {
  float lo = INFINITY, hi = -INFINITY;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < count;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const float v = static_cast<float>(x[i]);
    lo = fminf(lo, v);
    hi = fmaxf(hi, v);
  }
  __shared__ float sl[256], sh[256];
  sl[threadIdx.x] = lo;
  sh[threadIdx.x] = hi;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sl[threadIdx.x] = fminf(sl[threadIdx.x], sl[threadIdx.x + o]);
      sh[threadIdx.x] = fmaxf(sh[threadIdx.x], sh[threadIdx.x + o]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ws[2 * blockIdx.x] = sl[0];
    ws[2 * blockIdx.x + 1] = sh[0];
  }
}
__global__ void minmax_stage2_kernel(const float* __restrict__ ws, int nblocks, int x_bits, int x_sym,
                                     float* __restrict__ s_x, float* __restrict__ z_x) {
  if (threadIdx.x != 0) return;
  float lo = INFINITY, hi = -INFINITY;
  for (int i = 0; i < nblocks; ++i) {
    lo = fminf(lo, ws[2 * i]);
    hi = fmaxf(hi, ws[2 * i + 1]);
  }
  if (x_sym) {
    const double amax = fmax(fabs(static_cast<double>(lo)), fabs(static_cast<double>(hi)));
    float s = static_cast<float>(amax / static_cast<double>((1 << (x_bits - 1)) - 1));
    if (s == 0.f) s = 1.f;
    s_x[0] = s;
    z_x[0] = 0.f;
  } else {
    float s = static_cast<float>((static_cast<double>(hi) - static_cast<double>(lo)) /
                                 static_cast<double>((1 << x_bits) - 1));
    if (s == 0.f) s = 1.f;
    s_x[0] = s;
    z_x[0] = static_cast<float>(-rint(static_cast<double>(lo) / static_cast<double>(s)));
  }
}
void launch_minmax_act(const void* x, int dtype, int64_t count, int x_bits, int x_sym, float* s_x, float* z_x,
                       float* ws, cudaStream_t st) {
  const int g = grid_for(count, 256 * 8, 1024);
  count_launches(2);
  if (dtype == EFQAT_BF16)
    minmax_stage1_kernel<bf16><<<g, 256, 0, st>>>(static_cast<const bf16*>(x), count, ws);
  else
    minmax_stage1_kernel<float><<<g, 256, 0, st>>>(static_cast<const float*>(x), count, ws);
  minmax_stage2_kernel<<<1, 32, 0, st>>>(ws, g, x_bits, x_sym, s_x, z_x);
}

__global__ void __launch_bounds__(256) absmax_rows_kernel(const float* __restrict__ W, int64_t K, int w_bits,
                                                          float* __restrict__ s_w) {
  const int64_t n = blockIdx.x;
  float m = 0.f;
  for (int64_t k = threadIdx.x; k < K; k += blockDim.x) m = fmaxf(m, fabsf(W[n * K + k]));
  __shared__ float sh[256];
  sh[threadIdx.x] = m;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sh[threadIdx.x] = fmaxf(sh[threadIdx.x], sh[threadIdx.x + o]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    float s = static_cast<float>(static_cast<double>(sh[0]) / static_cast<double>((1 << (w_bits - 1)) - 1));
    if (s == 0.f) s = 1.f;
    s_w[n] = s;
  }
}
void launch_absmax_rows(const float* W, int64_t N, int64_t K, int w_bits, float* s_w, cudaStream_t st) {
  if (N == 0) return;
  count_launches(1);
  absmax_rows_kernel<<<static_cast<unsigned>(N), 256, 0, st>>>(W, K, w_bits, s_w);
}

}  // namespace efqat
