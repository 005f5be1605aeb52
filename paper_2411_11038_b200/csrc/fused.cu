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

// ---- job: weights -> bf16 operand (MODE 0 codes, MODE 1 dequantised) -------------------
// Flat over 8-element vectors (K % 8 == 0, so a vector never straddles two rows), four
// independent loads in flight per thread.
template <int MODE>
__device__ __forceinline__ void job_weights(const PrepArgs& a, int block, int nblocks) {
  const int64_t kv = a.K / 8;
  const int64_t nvec = a.N * kv;
  const int64_t stride = static_cast<int64_t>(nblocks) * blockDim.x;
  for (int64_t v0 = static_cast<int64_t>(block) * blockDim.x + threadIdx.x; v0 < nvec; v0 += 4 * stride) {
    float v[4][8];
    float sc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t i = v0 + u * stride;
      if (i < nvec) {
        ld8<float>(a.W + i * 8, v[u]);
        sc[u] = __ldg(a.s_w + i / kv);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t i = v0 + u * stride;
      if (i < nvec) {
        float sw = sc[u];
        if (!scale_ok(sw)) {
          record_status(a.status, EFQAT_DEV_BAD_SCALE);
          sw = 1.f;
        }
        const RowQ p = make_rowq(sw, a.w_bits);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float q = quant_weight(v[u][j], p).c0;
          v[u][j] = (MODE == 0) ? q : __fmul_rn(p.s, q);
        }
        st8(a.Wq + i * 8, v[u]);
      }
    }
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
  const int64_t stride = static_cast<int64_t>(nblocks) * blockDim.x;
  for (int64_t i0 = static_cast<int64_t>(block) * blockDim.x + threadIdx.x; i0 < n8; i0 += 4 * stride) {
    float v[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i0 + u * stride < n8) ld8<T>(X + (i0 + u * stride) * 8, v[u]);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u * stride < n8) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[u][j] = quant_act(v[u][j], p).c0;
        int64_t o = i0 + u * stride;
        if (a.xp_C8) {                     // pixel (b, h, w) goes to (b, h + pad, w + pad) of the padded image
          const int64_t px = o / a.xp_C8, c8 = o - px * a.xp_C8;
          const int64_t t = px / a.xp_W, w = px - t * a.xp_W;
          const int64_t b = t / a.xp_H, h = t - b * a.xp_H;
          const int64_t Wp = a.xp_W + 2 * a.xp_pad, Hp = a.xp_H + 2 * a.xp_pad;
          o = ((b * Hp + h + a.xp_pad) * Wp + w + a.xp_pad) * a.xp_C8 + c8;
        }
        st8(a.Xc + o * 8, v[u]);
      }
    }
  }
  if (a.xp_C8 && a.xp_pad > 0) {
    // the zero frame: 2 pad full rows, then 2 pad pixels at the ends of each of the H rows between
    const int64_t Wp = a.xp_W + 2 * a.xp_pad, Hp = a.xp_H + 2 * a.xp_pad;
    const int64_t full = 2 * a.xp_pad * Wp, side = 2 * a.xp_pad;
    const int64_t per_img = full + a.xp_H * side;
    const int64_t images = a.x_count / 8 / (static_cast<int64_t>(a.xp_C8) * a.xp_H * a.xp_W);
    const int64_t total = images * per_img * a.xp_C8;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t i = static_cast<int64_t>(block) * blockDim.x + threadIdx.x; i < total; i += stride) {
      const int64_t fp = i / a.xp_C8, c8 = i - fp * a.xp_C8;
      const int64_t b = fp / per_img, j = fp - b * per_img;
      int64_t hp, wp;
      if (j < full) {
        const int64_t r = j / Wp;
        hp = r < a.xp_pad ? r : Hp - 2 * a.xp_pad + r;
        wp = j - r * Wp;
      } else {
        const int64_t h = (j - full) / side, k = (j - full) - h * side;
        hp = h + a.xp_pad;
        wp = k < a.xp_pad ? k : a.xp_W + k;
      }
      *reinterpret_cast<uint4*>(a.Xc + (((b * Hp + hp) * Wp + wp) * a.xp_C8 + c8) * 8) = z;
    }
  }
}

// ---- jobs of the integer forward: 8-bit codes -------------------------------------------
__device__ __forceinline__ uint32_t pack4(const int (&c)[8], int o) {
  return (static_cast<uint32_t>(c[o]) & 255u) | ((static_cast<uint32_t>(c[o + 1]) & 255u) << 8) |
         ((static_cast<uint32_t>(c[o + 2]) & 255u) << 16) | ((static_cast<uint32_t>(c[o + 3]) & 255u) << 24);
}
// One warp per weight row: signed codes and their sum (the zero-point correction of the epilogue).
__device__ __forceinline__ void job_weights_i8(const PrepArgs& a, int block, int nblocks) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t kv = a.K / 8;
  for (int64_t n = static_cast<int64_t>(block) * 8 + warp; n < a.N; n += static_cast<int64_t>(nblocks) * 8) {
    float sw = __ldg(a.s_w + n);
    if (!scale_ok(sw)) {
      if (lane == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
      sw = 1.f;
    }
    const RowQ p = make_rowq(sw, a.w_bits);
    const float* row = a.W + n * a.K;
    int8_t* orow = a.Wq8 + n * a.K;
    int sum = 0;
    for (int64_t v0 = lane; v0 < kv; v0 += 128) {       // four independent 32-byte loads in flight
      float v[4][8];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (v0 + 32 * u < kv) ld8<float>(row + (v0 + 32 * u) * 8, v[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (v0 + 32 * u < kv) {
          int c[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            c[j] = quant_weight(v[u][j], p).code;
            sum += c[j];
          }
          *reinterpret_cast<uint2*>(orow + (v0 + 32 * u) * 8) = make_uint2(pack4(c, 0), pack4(c, 4));
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) a.wsum[n] = sum;
  }
}
// Activations -> 8-bit codes clamp(rne(x/s) + Zr, lo, hi) (unsigned; signed for the symmetric quantizer).
template <typename T>
__device__ __forceinline__ void job_quant_x_i8(const PrepArgs& a, int block, int nblocks) {
  bool bad;
  const ActQ p = make_actq(a.s_x, a.z_x, a.x_bits, a.x_sym, &bad);
  if (bad && block == 0 && threadIdx.x == 0) record_status(a.status, EFQAT_DEV_BAD_SCALE);
  const T* X = static_cast<const T*>(a.X);
  const int64_t n8 = a.x_count / 8;
  const int64_t stride = static_cast<int64_t>(nblocks) * blockDim.x;
  for (int64_t i0 = static_cast<int64_t>(block) * blockDim.x + threadIdx.x; i0 < n8; i0 += 4 * stride) {
    float v[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i0 + u * stride < n8) ld8<T>(X + (i0 + u * stride) * 8, v[u]);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u * stride < n8) {
        int c[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = quant_act(v[u][j], p).code;
        *reinterpret_cast<uint2*>(a.Xc8 + (i0 + u * stride) * 8) = make_uint2(pack4(c, 0), pack4(c, 4));
      }
    }
  }
}

// ---- job: one pass over dY: column-sum partials and the bf16 copy ------------------------
// Block (cb, slab): 256 columns x one slab of rows; warp w takes rows slab_lo + w, + 8, ...,
// four rows (four independent 16-byte loads per thread) at a time.
template <typename T>
__device__ __forceinline__ void job_dy_pass(const PrepArgs& a, int cb, int slab, float* sh /* [8][256] */) {
  const T* dY = static_cast<const T*>(a.dY);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // Narrow matrices (N a power of two up to 128): a row needs only N / 8 lanes, so a warp takes
  // 32 / (N / 8) rows per pass instead of leaving most of its lanes without a column.
  int lpr = 32;
  if (a.N <= 128 && (a.N & (a.N - 1)) == 0) lpr = static_cast<int>(a.N >> 3);
  const int R = 32 / lpr;                        // rows per warp and pass
  const int rs = lane / lpr, cl = lane - rs * lpr;
  const int64_t c0 = static_cast<int64_t>(cb) * 256 + cl * 8;
  const int64_t rows = ceil_div(a.M, static_cast<int64_t>(a.slabs));
  const int64_t m_lo = slab * rows;
  const int64_t m_hi = (m_lo + rows < a.M) ? m_lo + rows : a.M;
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  if (c0 < a.N) {
    for (int64_t m = m_lo + warp * R + rs; m < m_hi; m += 32 * R) {
      float v[4][8];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (m + 8 * R * u < m_hi) ld8<T>(dY + (m + 8 * R * u) * a.N + c0, v[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (m + 8 * R * u < m_hi) {
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] += v[u][j];
          if (a.dYb) st8(a.dYb + (m + 8 * R * u) * a.N + c0, v[u]);
        }
      }
    }
  }
  // the lanes that shared a column group add up (fixed order: reproducible)
  for (int off = lpr; off < 32; off <<= 1) {
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], off);
  }
  if (a.colsum_ws) {
    if (rs == 0) {
#pragma unroll
      for (int j = 0; j < 8; ++j) sh[warp * 256 + cl * 8 + j] = acc[j];
    }
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

// ---- job: gathered matrix dYsel[m, i] = bf16(dY[m, idx[i]]), pad columns [k_sel, pitch) zero ----
// Whole rows of the gathered matrix leave as full 128-byte lines.  Block `slab` covers the rows
// of that slab of the dY pass and sits next to the slab's column-sum blocks in launch order,
// so its scattered 2- or 4-byte reads of dY meet the same sectors in L2 (or in flight to it).
// The index list is staged in shared memory 1024 entries at a time.
template <typename T>
__device__ __forceinline__ void job_gather(const PrepArgs& a, int block, int32_t* s_idx /* [1024] */) {
  const T* dY = static_cast<const T*>(a.dY);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t rows = ceil_div(a.M, static_cast<int64_t>(a.slabs));
  const int64_t m_lo = block * rows;
  const int64_t m_hi = (m_lo + rows < a.M) ? m_lo + rows : a.M;
  for (int64_t ch = 0; ch < a.pitch; ch += 1024) {
    const int n = static_cast<int>((a.pitch - ch < 1024) ? a.pitch - ch : 1024);     // even: pitch % 16 == 0
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      int c = -1;
      if (ch + i < a.k_sel) {
        c = __ldg(a.idx + ch + i);
        // index contract: strictly ascending, inside [0, N)
        const bool bad = c < 0 || c >= a.N || (ch + i > 0 && __ldg(a.idx + ch + i - 1) >= c);
        if (bad) {
          if (block == 0) record_status(a.status, EFQAT_DEV_BAD_INDEX);
          c = -1;
        }
      }
      s_idx[i] = c;
    }
    __syncthreads();
    for (int64_t m = m_lo + warp; m < m_hi; m += 32) {        // four rows in flight per warp
      for (int i = 2 * lane; i < n; i += 64) {
        const int ca = s_idx[i], cb = s_idx[i + 1];
        float va[4], vb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int64_t r = m + 8 * u;
          va[u] = (r < m_hi && ca >= 0) ? static_cast<float>(dY[r * a.N + ca]) : 0.f;
          vb[u] = (r < m_hi && cb >= 0) ? static_cast<float>(dY[r * a.N + cb]) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int64_t r = m + 8 * u;
          if (r < m_hi) *reinterpret_cast<uint32_t*>(a.dYsel + r * a.pitch + ch + i) = pk2(va[u], vb[u]);
        }
      }
    }
  }
}

__device__ __forceinline__ void finalize_body(const FinArgs& a, const int b, double (*shd)[256], float4* red);

// Blocks [0, nb_prep) are the prepare jobs of one layer; blocks behind them (if any) are the
// finalize work of ANOTHER layer whose GEMMs have just completed: in a chain of layers the two
// are independent, and as one launch they cost one launch latency instead of two.
template <int W_MODE, typename TX>
__global__ void __launch_bounds__(256, 3) prepare_kernel(const PrepArgs a, const FinArgs f, const int nb_prep) {
  __shared__ __align__(16) float sh[8 * 256];
  pdl_trigger();
  pdl_wait();
  if (static_cast<int>(blockIdx.x) >= nb_prep) {
    finalize_body(f, static_cast<int>(blockIdx.x) - nb_prep, reinterpret_cast<double(*)[256]>(sh),
                  reinterpret_cast<float4*>(sh + 1024));
    return;
  }
  const int b = blockIdx.x;
  const int per_slab = a.col_blocks * a.dy_on + a.nb_g;
  const int nb_y = per_slab * a.slabs;
  if (b < nb_y) {
    // per slab of rows: [gather block,] then the column blocks of the dY pass.  These come first
    // in launch order: the gather blocks are the longest dependent chains of the launch, and
    // the short flat quantizer blocks behind them fill its tail.
    const int slab = b / per_slab, j = b - slab * per_slab;
    if (j < a.nb_g) job_gather<TX>(a, slab, reinterpret_cast<int32_t*>(sh));
    else job_dy_pass<TX>(a, j - a.nb_g, slab, sh);
  } else if (b < nb_y + a.nb_w) {
    if (W_MODE == 0 && a.i8) job_weights_i8(a, b - nb_y, a.nb_w);
    else job_weights<W_MODE>(a, b - nb_y, a.nb_w);
  } else {
    if (W_MODE == 0 && a.i8) job_quant_x_i8<TX>(a, b - nb_y - a.nb_w, a.nb_x);
    else job_quant_x<TX>(a, b - nb_y - a.nb_w, a.nb_x);
  }
}

// ---- finalize: dW rows (mask, dS_w, optional SGD) | dS_x, dZ_x | db ------------------------
// Block b of the finalize work of one layer; shd / red: 4 KiB of shared memory each.
__device__ __forceinline__ void finalize_body(const FinArgs& a, const int b, double (*shd)[256], float4* red) {
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
    // Short rows leave most of the block idle in the k loop, so the split partial products are
    // shared out over G groups of threads and combined through shared memory in a fixed order.
    const int nk4 = static_cast<int>(a.K >> 2);
    int G = 1;
    if (nk4 < 256) {
      G = 256 / nk4;
      if (G > a.splits) G = a.splits;
      if (G < 1) G = 1;
    }
    const int kq = (G > 1) ? static_cast<int>(threadIdx.x) % nk4 : static_cast<int>(threadIdx.x);
    const int sg = (G > 1) ? static_cast<int>(threadIdx.x) / nk4 : 0;
    double acc = 0.0;
    for (int64_t k0 = 0; k0 < a.K; k0 += 1024) {       // one pass unless K > 1024
      const int64_t k = k0 + 4 * kq;
      float4 g = make_float4(0.f, 0.f, 0.f, 0.f);
      if (k < a.K && sg < G) {
        for (int sp0 = sg; sp0 < a.splits; sp0 += 8 * G) {       // eight independent loads in flight
          float4 t[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            t[u] = (sp0 + u * G < a.splits)
                       ? __ldg(reinterpret_cast<const float4*>(a.P + (sp0 + u * G) * a.split_stride + i * a.K + k))
                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            g.x += t[u].x; g.y += t[u].y; g.z += t[u].z; g.w += t[u].w;
          }
        }
      }
      if (G > 1) {
        __syncthreads();
        red[threadIdx.x] = g;
        __syncthreads();
        if (sg == 0 && k < a.K) {
          for (int j = 1; j < G; ++j) {
            const float4 t = red[j * nk4 + kq];
            g.x += t.x; g.y += t.y; g.z += t.z; g.w += t.w;
          }
        }
      }
      if (sg == 0 && k < a.K) {
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
    const float2* pp = reinterpret_cast<const float2*>(a.dx_partials);
#pragma unroll 8
    for (int i = threadIdx.x; i < a.n_partials; i += 256) {
      const float2 t = pp[i];
      x += static_cast<double>(t.x);
      z += static_cast<double>(t.y);
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
    if (n < a.N) {
#pragma unroll 16
      for (int s = j; s < a.slabs; s += 8) acc += static_cast<double>(a.colsum_ws[static_cast<int64_t>(s) * a.N + n]);
    }
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

__global__ void __launch_bounds__(256) finalize_kernel(const FinArgs a) {
  __shared__ double shd[2][256];
  __shared__ float4 red[256];
  pdl_trigger();
  pdl_wait();
  finalize_body(a, blockIdx.x, shd, red);
}

}  // namespace

// Row slabs of the dY pass: blocks of 256 columns x one slab of rows, 64 rows (32 KiB of
// bf16) each until there are 512 slabs; beyond that the slabs grow, so that the sum over the
// slabs' column-sum partials stays short.
int prepare_slabs(int64_t M, int64_t N) {
  (void)N;
  int64_t s = ceil_div(M, 64);
  if (s > 512) s = 512;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}

// Blocks of a flat job: about `per_block` vectors of 8 elements each, at most four waves of the GPU.
static int flat_blocks(int64_t vectors, int64_t per_block) {
  int64_t nb = ceil_div(vectors, per_block);
  if (nb > 148 * 12) nb = 148 * 12;
  if (nb < 1) nb = 1;
  return static_cast<int>(nb);
}

static int finalize_blocks(const FinArgs& a) {
  const int nb_db = a.db ? static_cast<int>(ceil_div(a.N, 32)) : 0;
  return static_cast<int>(a.k_sel) + 1 + nb_db;
}

void launch_prepare(PrepArgs a, int w_mode, int act_bf16, cudaStream_t st, const FinArgs* fin) {
  a.nb_w = flat_blocks(a.N * (a.K / 8), 256 * 4);       // 32 KiB of fp32 weights per block
  if (a.i8) a.nb_w = static_cast<int>(ceil_div(a.N, 8) < 148 * 12 ? ceil_div(a.N, 8) : 148 * 12);   // a warp per row
  if (!a.W) a.nb_w = 0;                          // weight operand supplied by the layer's cache
  a.nb_x = 0;
  if (a.Xc || (a.i8 && a.Xc8)) a.nb_x = flat_blocks(a.x_count / 8, 256 * 8);   // 32 KiB (bf16) / 64 KiB (fp32) per block
  const bool gather = a.dY && a.dYsel && a.k_sel > 0 && a.k_sel < a.N;
  a.nb_g = gather ? 1 : 0;                       // gather blocks per slab
  a.col_blocks = static_cast<int>(ceil_div(a.N, 256));
  a.slabs = prepare_slabs(a.M, a.N);
  a.dy_on = (a.dY && (a.colsum_ws || a.dYb)) ? 1 : 0;
  const int nb_y = (a.col_blocks * a.dy_on + a.nb_g) * a.slabs;
  const int nb_prep = a.nb_w + a.nb_x + nb_y;
  const FinArgs f = fin ? *fin : FinArgs{};
  const int grid = nb_prep + (fin ? finalize_blocks(f) : 0);
  if (grid == 0) return;                         // cached weights, nothing unfrozen, no bias gradient wanted
  count_launches(1);
  if (w_mode == 0) {
    if (act_bf16) launch_dependent(prepare_kernel<0, bf16>, grid, 256, 0, st, 1, a, f, nb_prep);
    else launch_dependent(prepare_kernel<0, float>, grid, 256, 0, st, 1, a, f, nb_prep);
  } else {
    if (act_bf16) launch_dependent(prepare_kernel<1, bf16>, grid, 256, 0, st, 1, a, f, nb_prep);
    else launch_dependent(prepare_kernel<1, float>, grid, 256, 0, st, 1, a, f, nb_prep);
  }
}

void launch_finalize(FinArgs a, cudaStream_t st) {
  const int grid = finalize_blocks(a);
  count_launches(1);
  launch_dependent(finalize_kernel, grid, 256, 0, st, 1, a);
}

}  // namespace efqat
