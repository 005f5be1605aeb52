// Bandwidth-class kernels outside the fused prepare / finalize launches: quantizer export
// (codes and clip flags), the stand-alone column sums of dY, MinMax initialisation.
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

static int grid_for(int64_t work_items, int threads, int max_blocks = 148 * 16) {
  int64_t b = ceil_div(work_items, threads);
  if (b < 1) b = 1;
  if (b > max_blocks) b = max_blocks;
  return static_cast<int>(b);
}

// ------------------------------------------------------------------ activation quantizer
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
