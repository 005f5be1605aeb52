// Fused bandwidth-class kernels of the layer step: one "prepare" launch in front of the
// GEMMs and one "finalize" launch behind them, each covering several independent jobs
// through block ranges, so that a forward is 2 launches and a backward 4.
#include "internal.h"

namespace efqat {

namespace {

template <typename T>
__device__ __forceinline__ void ld8(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void ld8<float>(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <>
__device__ __forceinline__ void ld8<bf16>(const bf16* p, float (&v)[8]) {
  const uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint32_t pk2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void st8(bf16* p, const float (&v)[8]) {
  uint4 o;
  o.x = pk2(v[0], v[1]); o.y = pk2(v[2], v[3]); o.z = pk2(v[4], v[5]); o.w = pk2(v[6], v[7]);
  *reinterpret_cast<uint4*>(p) = o;
}

// ---- job: weight rows -> bf16 operand (MODE 0 codes, MODE 1 dequantised) --------------
template <int MODE>
__device__ __forceinline__ void job_weight_row(const PrepArgs& a, int64_t n) {
  float s = a.s_w[n];
  if (!scale_ok(s)) {
    if (threadIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
    s = 1.f;
  }
  const RowQ p = make_rowq(s, a.w_bits);
  const float* row = a.W + n * a.K;
  bf16* orow = a.Wq + n * a.K;
  for (int64_t k = threadIdx.x * 8; k < a.K; k += blockDim.x * 8) {
    float v[8];
    ld8<float>(row + k, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float q = quant_weight(v[j], p).c0;
      v[j] = (MODE == 0) ? q : __fmul_rn(p.s, q);
    }
    st8(orow + k, v);
  }
}

// ---- job: activations -> centred integer codes as bf16 --------------------------------
template <typename T>
__device__ __forceinline__ void job_quant_x(const PrepArgs& a, int block, int nblocks) {
  bool bad;
  const ActQ p = make_actq(a.s_x, a.z_x, a.x_bits, a.x_sym, &bad);
  if (bad && block == 0 && threadIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
  const T* X = static_cast<const T*>(a.X);
  const int64_t n8 = a.x_count / 8;
  for (int64_t i = static_cast<int64_t>(block) * blockDim.x + threadIdx.x; i < n8;
       i += static_cast<int64_t>(nblocks) * blockDim.x) {
    float v[8];
    ld8<T>(X + i * 8, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = quant_act(v[j], p).c0;
    st8(a.Xc + i * 8, v);
  }
}

// ---- job: one pass over dY: column-sum partials, gather of the selected columns, bf16 copy
// Block (cb, slab): 256 columns x one slab of rows; warp w takes rows slab_lo + w, + 8, ...
template <typename T>
__device__ __forceinline__ void job_dy_pass(const PrepArgs& a, int cb, int slab, float* sh /* [8][256] */) {
  const T* dY = static_cast<const T*>(a.dY);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t c0 = static_cast<int64_t>(cb) * 256 + lane * 8;
  const int64_t rows = ceil_div(a.M, static_cast<int64_t>(a.slabs));
  const int64_t m_lo = slab * rows;
  const int64_t m_hi = (m_lo + rows < a.M) ? m_lo + rows : a.M;
  const bool col_ok = c0 < a.N;
  const bool gather = a.k_sel > 0 && a.k_sel < a.N;
  int pos[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) pos[j] = -1;
  if (gather) {
    // Compact position of each of this thread's 8 consecutive columns in the ascending idx:
    // one binary search for the first column, then a merge walk.  The slice of idx that this
    // block's 256 columns can hit is staged in shared memory first (it holds at most 256 entries).
    __shared__ int s_lo, s_cnt;
    __shared__ int32_t s_idx[256];
    if (threadIdx.x == 0) {
      const int cfirst = cb * 256;
      int lo = 0, hi = static_cast<int>(a.k_sel);
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (a.idx[mid] < cfirst) lo = mid + 1; else hi = mid;
      }
      s_lo = lo;
      int l2 = lo, h2 = static_cast<int>(a.k_sel);
      while (l2 < h2) {
        const int mid = (l2 + h2) >> 1;
        if (a.idx[mid] < cfirst + 256) l2 = mid + 1; else h2 = mid;
      }
      s_cnt = (l2 - lo > 256) ? 256 : l2 - lo;      // more than 256 only for a broken (non-ascending) idx
    }
    __syncthreads();
    if (threadIdx.x < s_cnt) s_idx[threadIdx.x] = a.idx[s_lo + threadIdx.x];
    __syncthreads();
    if (col_ok) {
      int lo = 0, hi = s_cnt;
      const int cmin = static_cast<int>(c0);
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_idx[mid] < cmin) lo = mid + 1; else hi = mid;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (lo < s_cnt && s_idx[lo] == cmin + j) {
          pos[j] = s_lo + lo;
          ++lo;
        }
      }
    }
  }
  if (gather && cb == 0 && slab == 0) {
    // index contract: strictly ascending, inside [0, N)
    for (int j = threadIdx.x; j < a.k_sel; j += blockDim.x) {
      const int c = a.idx[j];
      if (c < 0 || c >= a.N || (j > 0 && a.idx[j - 1] >= c)) record_status(a.status, EFQAT_DEV_BAD_INDEX);
    }
  }
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  if (col_ok) {
    int64_t m = m_lo + warp;
    for (; m + 24 < m_hi; m += 32) {       // four independent 16-byte loads in flight per thread
      float v[4][8];
#pragma unroll
      for (int u = 0; u < 4; ++u) ld8<T>(dY + (m + 8 * u) * a.N + c0, v[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] += v[u][j];
        if (a.dYb) st8(a.dYb + (m + 8 * u) * a.N + c0, v[u]);
        if (gather) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (pos[j] >= 0) a.dYsel[(m + 8 * u) * a.pitch + pos[j]] = __float2bfloat16_rn(v[u][j]);
        }
      }
    }
    for (; m < m_hi; m += 8) {
      float v[8];
      ld8<T>(dY + m * a.N + c0, v);
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] += v[j];
      if (a.dYb) st8(a.dYb + m * a.N + c0, v);
      if (gather) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (pos[j] >= 0) a.dYsel[m * a.pitch + pos[j]] = __float2bfloat16_rn(v[j]);
      }
    }
  }
  if (gather && cb == 0) {
    // zero the pad columns [k_sel, pitch) of this slab's rows
    const int pad = static_cast<int>(a.pitch - a.k_sel);
    for (int64_t i = threadIdx.x; i < (m_hi - m_lo) * pad; i += blockDim.x)
      a.dYsel[(m_lo + i / pad) * a.pitch + a.k_sel + (i % pad)] = __float2bfloat16_rn(0.f);
  }
  if (a.colsum_ws) {
#pragma unroll
    for (int j = 0; j < 8; ++j) sh[warp * 256 + lane * 8 + j] = acc[j];
    __syncthreads();
    const int64_t c = static_cast<int64_t>(cb) * 256 + threadIdx.x;
    if (c < a.N) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += sh[w * 256 + threadIdx.x];
      a.colsum_ws[static_cast<int64_t>(slab) * a.N + c] = t;
    }
  }
}

template <int W_MODE, typename TX>
__global__ void __launch_bounds__(256, 3) prepare_kernel(const PrepArgs a) {
  __shared__ float sh[8 * 256];
  const int b = blockIdx.x;
  if (b < a.nb_w) {
    job_weight_row<W_MODE>(a, b);
  } else if (b < a.nb_w + a.nb_x) {
    job_quant_x<TX>(a, b - a.nb_w, a.nb_x);
  } else {
    const int r = b - a.nb_w - a.nb_x;
    job_dy_pass<TX>(a, r % a.col_blocks, r / a.col_blocks, sh);
  }
}

// ---- finalize: dW rows (mask, dS_w, optional SGD) | dS_x, dZ_x | db ------------------------
__global__ void __launch_bounds__(256) finalize_kernel(const FinArgs a) {
  __shared__ double shd[2][256];
  const int b = blockIdx.x;
  if (b < a.k_sel) {
    const int64_t i = b;
    const int64_t n = a.idx ? static_cast<int64_t>(a.idx[i]) : i;
    if (n < 0 || n >= a.N) {
      if (threadIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_INDEX);
      return;
    }
    float s = a.s_w[n];
    if (!scale_ok(s)) s = 1.f;    // reported by the prepare launch of the same call
    const RowQ p = make_rowq(s, a.w_bits);
    float sx = a.s_x[0];
    if (!scale_ok(sx)) sx = 1.f;
    const float* wrow = a.W + n * a.K;
    double acc = 0.0;
    for (int64_t k = threadIdx.x * 4; k < a.K; k += blockDim.x * 4) {
      float4 g = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp = 0; sp < a.splits; ++sp) {
        const float4 t = *reinterpret_cast<const float4*>(a.P + sp * a.split_stride + i * a.K + k);
        g.x += t.x; g.y += t.y; g.z += t.z; g.w += t.w;
      }
      const float4 w4 = *reinterpret_cast<const float4*>(wrow + k);
      const float gv[4] = {g.x * sx, g.y * sx, g.z * sx, g.w * sx};
      const float wv[4] = {w4.x, w4.y, w4.z, w4.w};
      float ov[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const QElem e = quant_weight(wv[j], p);
        ov[j] = e.flag ? 0.f : gv[j];
        acc += static_cast<double>(gv[j]) * static_cast<double>(e.t);
      }
      *reinterpret_cast<float4*>(a.dW_sel + i * a.K + k) = make_float4(ov[0], ov[1], ov[2], ov[3]);
      if (a.has_opt) {
        const int64_t o = n * a.K + k;
        const float4 w0 = *reinterpret_cast<const float4*>(a.opt.W_inout + o);
        const float4 m0 = *reinterpret_cast<const float4*>(a.opt.mom_inout + o);
        const float wi[4] = {w0.x, w0.y, w0.z, w0.w}, mi[4] = {m0.x, m0.y, m0.z, m0.w};
        float wo[4], mo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          mo[j] = a.opt.momentum * mi[j] + (ov[j] + a.opt.weight_decay * wi[j]);
          wo[j] = wi[j] - a.opt.lr * mo[j];
        }
        *reinterpret_cast<float4*>(a.opt.mom_inout + o) = make_float4(mo[0], mo[1], mo[2], mo[3]);
        *reinterpret_cast<float4*>(a.opt.W_inout + o) = make_float4(wo[0], wo[1], wo[2], wo[3]);
      }
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) shd[0][threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int w = 0; w < 8; ++w) t += shd[0][w];
      a.dS_w_sel[i] = static_cast<float>(t);
    }
  } else if (b == a.k_sel) {
    double x = 0.0, z = 0.0;
    for (int i = threadIdx.x; i < a.n_partials; i += 256) {
      x += static_cast<double>(a.dx_partials[2 * i]);
      z += static_cast<double>(a.dx_partials[2 * i + 1]);
    }
    shd[0][threadIdx.x] = x;
    shd[1][threadIdx.x] = z;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
      if (threadIdx.x < o) {
        shd[0][threadIdx.x] += shd[0][threadIdx.x + o];
        shd[1][threadIdx.x] += shd[1][threadIdx.x + o];
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      a.dS_x[0] = static_cast<float>(shd[0][0]);
      a.dZ_x[0] = static_cast<float>(shd[1][0]);
    }
  } else {
    // db: 32 columns per block, 8 threads per column over the slabs, fixed combination order
    const int c = threadIdx.x & 31, j = threadIdx.x >> 5;
    const int64_t n = static_cast<int64_t>(b - a.k_sel - 1) * 32 + c;
    double acc = 0.0;
    if (n < a.N)
      for (int s = j; s < a.slabs; s += 8) acc += static_cast<double>(a.colsum_ws[static_cast<int64_t>(s) * a.N + n]);
    shd[0][threadIdx.x] = acc;
    __syncthreads();
    if (j == 0 && n < a.N) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += shd[0][w * 32 + c];
      a.db[n] = static_cast<float>(t);
    }
  }
}

}  // namespace

// Row slabs of the dY pass: enough blocks (column blocks x slabs) to fill the GPU about four
// times over, at least 32 rows per slab.
int prepare_slabs(int64_t M, int64_t N) {
  const int64_t col_blocks = ceil_div(N, 256);
  int64_t s = ceil_div(4 * 148, col_blocks);
  const int64_t by_rows = ceil_div(M, 32);
  if (s > by_rows) s = by_rows;
  if (s > 2048) s = 2048;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}

void launch_prepare(PrepArgs a, int w_mode, int act_bf16, cudaStream_t st) {
  a.nb_w = static_cast<int>(a.N);
  a.nb_x = 0;
  if (a.Xc) {
    int64_t nb = ceil_div(a.x_count / 8, 256 * 2);
    if (nb > 148 * 8) nb = 148 * 8;
    if (nb < 1) nb = 1;
    a.nb_x = static_cast<int>(nb);
  }
  const bool gather = a.k_sel > 0 && a.k_sel < a.N;
  int nb_y = 0;
  a.col_blocks = static_cast<int>(ceil_div(a.N, 256));
  a.slabs = prepare_slabs(a.M, a.N);
  if (a.dY && (a.colsum_ws || gather || a.dYb)) nb_y = a.col_blocks * a.slabs;
  const int grid = a.nb_w + a.nb_x + nb_y;
  count_launches(1);
  if (w_mode == 0) {
    if (act_bf16) prepare_kernel<0, bf16><<<grid, 256, 0, st>>>(a);
    else prepare_kernel<0, float><<<grid, 256, 0, st>>>(a);
  } else {
    if (act_bf16) prepare_kernel<1, bf16><<<grid, 256, 0, st>>>(a);
    else prepare_kernel<1, float><<<grid, 256, 0, st>>>(a);
  }
}

void launch_finalize(FinArgs a, cudaStream_t st) {
  const int nb_db = a.db ? static_cast<int>(ceil_div(a.N, 32)) : 0;
  const int grid = static_cast<int>(a.k_sel) + 1 + nb_db;
  count_launches(1);
  finalize_kernel<<<grid, 256, 0, st>>>(a);
}

}  // namespace efqat
