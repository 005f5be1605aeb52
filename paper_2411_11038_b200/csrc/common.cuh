// Shared definitions of the CUDA path: the derived quantizer parameters and the
// per-element quantizer arithmetic (Eq. 1 and Eq. 3 of the paper).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/efqat.h"

namespace efqat {

// Derived per-tensor activation quantizer parameters, written once per call by
// prep_act_kernel and read by every kernel that quantizes activations.
struct ActQ {
  float s;        // scale
  float rinv;     // fl32(1/s): the multiplier that decides the integer code
  float rinv_lo;  // 1/s - rinv in fp32: correction term for the scale gradient
  float zr;       // rounded, clamped zero point (0 for the symmetric variant)
  float lo, hi;   // code range [lo, hi]
  float pad0, pad1;
};

struct QElem {
  float c0;   // clamp(c, lo, hi) - zr : the centred integer entering the contractions
  float t;    // d(dequantised value)/d(scale) under the straight-through estimator
  int flag;   // 0 in range, 1 clipped low, 2 clipped high
  int code;   // clamp(c, lo, hi)
};

// Programmatic dependent launch: every kernel of the layer path lets the next launch of the
// stream start early (pdl_trigger) and waits for the launches before it to finish, with
// their writes visible, before it touches global memory (pdl_wait).  Between the two, only
// set-up that reads no global data may run.  Both are no-ops for a plain launch.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void record_status(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// Round to nearest, ties to even, through the 1.5 * 2^23 constant: equal to rintf() for
// |u| < 2^22 and still far outside every code range beyond that, at two full-rate adds
// (rintf goes through the quarter-rate conversion unit).
__device__ __forceinline__ float rne_small(float u) {
  return __fadd_rn(__fadd_rn(u, 12582912.f), -12582912.f);
}

// Eq. 1 on one element.  The code is decided by u = fl32(x * fl32(1/s)), rounded to
// nearest-even; the scale gradient uses x/s to roughly fp64 accuracy through the
// two-term reciprocal (rne(u) - x*rinv is exact in one fma because rne(u) is within
// half a unit of the product).
__device__ __forceinline__ QElem quant_act(float x, const ActQ& p) {
  QElem e;
  const float u = __fmul_rn(x, p.rinv);
  const float r = rne_small(u);
  const float c = r + p.zr;
  const float q = fminf(fmaxf(c, p.lo), p.hi);
  e.flag = (c < p.lo) ? 1 : ((c > p.hi) ? 2 : 0);
  e.c0 = q - p.zr;
  e.code = static_cast<int>(q);
  // in range: t = rne(u) - x/s ; clipped: t = c0
  const float resid = fmaf(-x, p.rinv_lo, fmaf(-x, p.rinv, r));
  e.t = e.flag ? e.c0 : resid;
  return e;
}

// Derived activation-quantizer constants from the learnable scale / zero point.  A scale
// that is not positive and finite is replaced by 1 (and reported through *bad).
__device__ __forceinline__ ActQ make_actq(const float* __restrict__ s_x, const float* __restrict__ z_x,
                                          int x_bits, int x_sym, bool* bad) {
  ActQ p;
  float s = s_x[0];
  const bool ok = s > 0.f && isfinite(s);
  if (bad) *bad = !ok;
  if (!ok) s = 1.f;
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
  return p;
}

struct RowQ {
  float s, rinv, rinv_lo, qmax;
};

__device__ __forceinline__ RowQ make_rowq(float s, int w_bits) {
  RowQ r;
  r.s = s;
  const double inv = 1.0 / static_cast<double>(s);
  r.rinv = static_cast<float>(inv);
  r.rinv_lo = static_cast<float>(inv - static_cast<double>(r.rinv));
  r.qmax = static_cast<float>((1 << (w_bits - 1)) - 1);
  return r;
}

// Eq. 3 on one element (symmetric, zero point 0, clamp to [-qmax, qmax]).
__device__ __forceinline__ QElem quant_weight(float w, const RowQ& p) {
  QElem e;
  const float u = __fmul_rn(w, p.rinv);
  const float c = rne_small(u);
  const float q = fminf(fmaxf(c, -p.qmax), p.qmax);
  e.flag = (c < -p.qmax) ? 1 : ((c > p.qmax) ? 2 : 0);
  e.c0 = q;
  e.code = static_cast<int>(q);
  const float resid = fmaf(-w, p.rinv_lo, fmaf(-w, p.rinv, c));
  e.t = e.flag ? q : resid;
  return e;
}

__device__ __forceinline__ bool scale_ok(float s) { return s > 0.f && isfinite(s); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
__host__ __device__ inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

}  // namespace efqat
