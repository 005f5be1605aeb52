// Optimizer step of the quantization parameters (Section 4 "Setup": Adam for the quantization
// parameters; Algorithm 1: "update the unfrozen weight channels and their scales", "update the
// scales and zero points of the activations"), one launch per layer: the weight scales of the
// unfrozen channels, the activation scale and the activation zero point.  Appendix A.2's log2
// parameterisation optimises theta = log2(s) for the scales (gradient s * ln 2 * dL/ds through
// s = 2^theta) and keeps the zero point raw.
#include "internal.h"

namespace efqat {

namespace {

struct AdamConst {
  float lr, b1, b2, eps, inv_bc1, inv_bc2;
  int log2_scale;
};

// One Adam step on a single parameter; *theta is only touched in log2 mode.
__device__ __forceinline__ void adam_one(const AdamConst& c, bool log2_mode, float g, float* p, float* m, float* v,
                                         float* theta) {
  const float p0 = *p;
  if (log2_mode) g = g * p0 * 0.693147180559945309f;
  const float m1 = fmaf(c.b1, *m, (1.f - c.b1) * g);
  const float v1 = fmaf(c.b2, *v, (1.f - c.b2) * g * g);
  *m = m1;
  *v = v1;
  const float upd = c.lr * (m1 * c.inv_bc1) / (sqrtf(v1 * c.inv_bc2) + c.eps);
  if (log2_mode) {
    const float t1 = *theta - upd;
    *theta = t1;
    *p = exp2f(t1);
  } else {
    *p = p0 - upd;
  }
}

__global__ void __launch_bounds__(256) qparam_adam_kernel(AdamConst c, efqat_qparam_state st, int64_t N,
                                                          const int32_t* __restrict__ idx, int64_t k_sel,
                                                          const float* __restrict__ dS_w_sel,
                                                          const float* __restrict__ dS_x,
                                                          const float* __restrict__ dZ_x, int* status) {
  pdl_trigger();
  pdl_wait();
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < k_sel) {
    const int64_t n = idx ? static_cast<int64_t>(idx[i]) : i;
    if (n < 0 || n >= N) {
      record_status(status, EFQAT_DEV_BAD_INDEX);
      return;
    }
    adam_one(c, c.log2_scale != 0, dS_w_sel[i], st.s_w + n, st.m_sw + n, st.v_sw + n,
             c.log2_scale ? st.theta_sw + n : nullptr);
  } else if (i == k_sel) {
    adam_one(c, c.log2_scale != 0, dS_x[0], st.s_x, st.state_x + 0, st.state_x + 1, st.state_x + 4);
  } else if (i == k_sel + 1 && dZ_x) {
    adam_one(c, false, dZ_x[0], st.z_x, st.state_x + 2, st.state_x + 3, nullptr);
  }
}

__global__ void log2_init_kernel(const float* __restrict__ s, float* __restrict__ theta, int64_t n, int* status) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = s[i];
  if (!scale_ok(v)) record_status(status, EFQAT_DEV_BAD_SCALE);
  theta[i] = log2f(scale_ok(v) ? v : 1.f);
}

}  // namespace

void launch_qparam_adam(const efqat_adam& a, const efqat_qparam_state& st, int64_t N, const int32_t* idx,
                        int64_t k_sel, const float* dS_w_sel, const float* dS_x, const float* dZ_x, int* status,
                        cudaStream_t stream) {
  AdamConst c;
  c.lr = a.lr; c.b1 = a.beta1; c.b2 = a.beta2; c.eps = a.eps;
  // bias corrections 1 - beta^t in double on the host
  c.inv_bc1 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(a.beta1), static_cast<double>(a.step))));
  c.inv_bc2 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(a.beta2), static_cast<double>(a.step))));
  c.log2_scale = a.log2_scale;
  const unsigned grid = static_cast<unsigned>(ceil_div(k_sel + 2, 256));
  count_launches(1);
  launch_dependent(qparam_adam_kernel, grid, 256, 0, stream, 1, c, st, N, idx, k_sel, dS_w_sel, dS_x, dZ_x, status);
}

void launch_log2_init(const float* s, float* theta, int64_t n, int* status, cudaStream_t stream) {
  count_launches(1);
  log2_init_kernel<<<static_cast<unsigned>(ceil_div(n, 256)), 256, 0, stream>>>(s, theta, n, status);
}

}  // namespace efqat
