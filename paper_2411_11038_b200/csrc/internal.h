// Host-side launchers shared between the translation units of the library.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace efqat {

typedef __nv_bfloat16 bf16;

// Adds n to the launch counter of the context whose entry point is running on this thread
// (reported by efqat_launch_count); a no-op outside an entry point that has a context.
void count_launches(int n);
// Bounded-wait self-test (selftest.cu): one mbarrier nobody arrives on, waited for limit_ns.
void launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st);

// Launch with programmatic stream serialization: the kernel may begin while the previous
// launch of the stream drains; it must call pdl_wait() before reading or writing global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                    unsigned cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n = 0;
  at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = cluster_x;
    at[n].val.clusterDim.y = 1;
    at[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// ---- elementwise.cu -----------------------------------------------------------------
void launch_prep_act(const float* s_x, const float* z_x, int x_bits, int x_sym, ActQ* out, int* status,
                     cudaStream_t st);
void launch_quant_act_export(const void* X, int dtype, int64_t count, const ActQ* q, int32_t* codes,
                             uint8_t* clip, cudaStream_t st);
void launch_quant_weight_export(const float* W, int64_t N, int64_t K, const float* s_w, int w_bits,
                                int32_t* codes, uint8_t* clip, int* status, cudaStream_t st);
// ws: COLSUM_SLABS * N floats
static const int COLSUM_SLABS = 64;
void launch_colsum(const void* dY, int dtype, int64_t M, int64_t N, float* ws, float* db, cudaStream_t st);
void launch_minmax_act(const void* x, int dtype, int64_t count, int x_bits, int x_sym, float* s_x, float* z_x,
                       float* ws, cudaStream_t st);
void launch_absmax_rows(const float* W, int64_t N, int64_t K, int w_bits, float* s_w, cudaStream_t st);

// ---- fused.cu -----------------------------------------------------------------------
// One launch in front of the GEMMs: weight rows -> bf16 operand, activations -> centred codes
// (skipped when Xc is null), one pass over dY (skipped when dY is null or nothing of it is
// wanted) producing column-sum partials and a bf16 copy, and the gather of the selected
// columns of dY (when dYsel is set and 0 < k_sel < N).
struct PrepArgs {
  int64_t M, N, K;
  const float* W; const float* s_w; int w_bits; bf16* Wq;
  const void* X; const float* s_x; const float* z_x; int x_bits, x_sym; bf16* Xc;
  int64_t x_count;   // elements of X (B*H*W*Cin for convolutions, M*K otherwise)
  // Padded code layout (convolutions with few input channels): Xc is [B, xp_H + 2 pad, xp_W + 2 pad, 8 xp_C8]
  // with the quantized pixel (h, w) at (h + pad, w + pad) and zeros around it.  xp_C8 == 0: dense.
  int xp_C8, xp_H, xp_W, xp_pad;
  const void* dY; bf16* dYb; float* colsum_ws;
  const int32_t* idx; int64_t k_sel, pitch; bf16* dYsel;
  int* status;
  // forward on the integer tensor cores: 8-bit codes (weights signed, activations unsigned or,
  // for the symmetric quantizer, signed; not centred) and the row sums of the weight codes
  int i8; int8_t* Wq8; uint8_t* Xc8; int32_t* wsum;
  int nb_g, nb_w, nb_x, col_blocks, slabs, dy_on;   // filled by launch_prepare
};
int prepare_slabs(int64_t M, int64_t N);

// One launch behind the GEMMs: dW rows (split reduction, clip mask, dS_w, optional SGD),
// dS_x / dZ_x from the per-tile partials, db from the column-sum partials.
struct FinArgs {
  int64_t N, K, k_sel;
  const float* P; int splits; int64_t split_stride;
  const float* W; const float* s_w; const float* s_x; int w_bits;
  const int32_t* idx;
  float* dW_sel; float* dS_w_sel;
  efqat_sgd opt; int has_opt;
  const float* dx_partials; int n_partials; float* dS_x; float* dZ_x;
  const float* colsum_ws; int slabs; float* db;
  int* status;
};
void launch_finalize(FinArgs a, cudaStream_t st);
// fin != null: the finalize work of another layer rides behind the prepare jobs in the same launch
void launch_prepare(PrepArgs a, int w_mode, int act_bf16, cudaStream_t st, const FinArgs* fin = nullptr);

// ---- optim.cu -----------------------------------------------------------------------
void launch_qparam_adam(const efqat_adam& a, const efqat_qparam_state& st, int64_t N, const int32_t* idx,
                        int64_t k_sel, const float* dS_w_sel, const float* dS_x, const float* dZ_x, int* status,
                        cudaStream_t stream);
void launch_log2_init(const float* s, float* theta, int64_t n, int* status, cudaStream_t stream);

// ---- cache.cu -----------------------------------------------------------------------
// Rebuilds rows of a layer's weight-operand cache: rows idx[0..rows) (idx null: rows 0..rows).
// codes8 + wsum (integer forward) or codes16 (bf16 forward) and what (backward) as laid out
// by the cache carving of the entry points.
struct CacheArgs {
  int64_t N, K, rows;
  const float* W; const float* s_w; int w_bits;
  const int32_t* idx;
  int8_t* codes8; int32_t* wsum; bf16* codes16; bf16* what;
  int* status;
};
void launch_weight_cache(const CacheArgs& a, cudaStream_t st);

// ---- skinny.cu ----------------------------------------------------------------------
// Forward of a plain layer with a contraction of 64 or 128 in one launch: fake-quant of X as the
// operand producer, weight codes resident in shared memory, epilogue straight to global memory.
// W (fp32, quantized in the kernel) or codes16 (the layer cache's bf16 codes) supplies the weights.
bool skinny_fwd_applies(int64_t M, int64_t N, int64_t K, int act_bf16);
int run_skinny_fwd(int64_t M, int64_t N, int64_t K, int act_bf16, const void* X, void* Y, const float* W,
                   const bf16* codes16, const float* s_w, const float* s_x, const float* z_x, const float* bias,
                   int w_bits, int x_bits, int x_sym, int* status, int sm_count, cudaStream_t st);

// ---- skinny_bwd.cu ------------------------------------------------------------------
// Backward of a plain bf16 layer with K = 64 and N = 128 or 256 in one pass over dY and X: grad
// input with the STE epilogue, the weight-gradient partial of every CTA (rows of the channels idx
// only: P [grid][k_sel][64], raw sums) and the column sums of dY (colsum [grid][N], may be null),
// dS_x / dZ_x partials (dxpart [grid * 8][2]); grid = skinny_bwd_grid().  The finalize launch
// sums the per-CTA partials (splits = slabs = grid).  W (fp32) or what (cached bf16 W^) supplies
// the weights.
bool skinny_bwd_applies(int64_t M, int64_t N, int64_t K, int act_bf16);
int skinny_bwd_grid(int64_t M, int sm_count);
int run_skinny_bwd(int64_t M, int64_t N, const void* dY, const void* X, void* dX, const float* W, const bf16* what,
                   const float* s_w, int w_bits, const float* s_x, const float* z_x, int x_bits, int x_sym,
                   const int32_t* idx, int64_t k_sel, float* P, float* colsum, float* dxpart, int* status,
                   int sm_count, cudaStream_t st);

// ---- select.cu ----------------------------------------------------------------------
size_t select_workspace_bytes(int L, int64_t total_channels);
int run_select(int mode, int L, const efqat_layer_desc* layers, const float* const* weights, const int64_t* k,
               int32_t* idx, int32_t* offsets, float* importance, void* ws, size_t ws_bytes, int* status,
               cudaStream_t st);

// ---- gemm.cu ------------------------------------------------------------------------
enum GemmEpi { EPI_FWD = 0, EPI_DX = 1, EPI_PART = 2, EPI_FWD_I8 = 3 };   // EPI_FWD_I8: chosen inside run_gemm

// Implicit-GEMM convolution geometry (stride 1 or 2).  The activation operand is read through a
// 4-D tensor map over its NHWC tensor with a box of pixels shifted by the filter tap; pixels
// that fall into the padding come back as zeros from the TMA unit, and so do channels past the
// tensor's last one (channel counts that are not multiples of 64).
//   mode 1 forward : A = Xc [B,H,W,Cin] patches, B = weight codes [N, R*S*Cin], D = Y [B,Ho,Wo,N]
//   mode 2 grad-in : A = dY [B,Ho,Wo,N] patches, B = W^ [N, R*S*Cin] (MN-major), D = dX [B,H,W,Cin]
//   mode 3 grad-w  : A = Xc patches (MN-major), B = gathered dY [B,Ho,Wo,pitch] (MN-major),
//                    D[(r,s,c), i] partial products, contraction over output pixels
// A view of an NHWC tensor as W x H pixels per image with explicit pitches (elements).
struct ConvView { const void* base; int64_t W, H, pix, row, img; };
// A grad-input launch (mode 2) described directly instead of through (R, S, pad, stride, class):
// the pixel space it tiles, its filter taps and the views of dY (by tap_map), of dX and of X.
struct ConvExplicit {
  int pW, pH;                       // pixel space of the launch (images: ConvArgs::B); columns of D: GemmArgs::Nc
  int ntaps;
  int8_t tap_dh[49], tap_dw[49];    // tap t reads the dY view tap_map[t] shifted by (tap_dw, tap_dh) pixels
  uint8_t tap_map[49], tap_rs[49];  // ... against columns [64 tap_rs[t], 64 tap_rs[t] + Nc) of the B matrix
  ConvView a_view[4];
  const void* x_base;               // dX (GemmArgs::out) and X share the pitches of o_view; X starts here
  ConvView o_view;
  int64_t b_cols;                   // columns (row pitch) of the B matrix [N, b_cols]
};

// Strip form of the grad-input of a convolution with few input channels (P = 64 / Cin input pixels
// of one row are one output row of the GEMM): the banded weight matrix T [N, R * nP * 64] built
// from the dequantised weights what [N, R * S * Cin]; nP = number of output columns p_min .. that
// reach a strip.
struct StripArgs {
  const bf16* what; bf16* T;
  int64_t N;
  int R, S, Cin, pad, stride, p_min, nP;
};
void launch_strip_weights(const StripArgs& a, cudaStream_t st);

struct ConvArgs {
  const ConvExplicit* ex;           // null: derived from the fields below
  int mode;
  int B, H, W, Cin;     // input activation tensor
  int Ho, Wo, N;        // output activation tensor
  int R, S, pad;
  int stride;           // 1 or 2
  // mode 2 only: the class of input pixels (cls_h + stride * i, cls_w + stride * j) this launch
  // computes; a strided grad-input is one launch per class, each with the taps that reach it
  int cls_h, cls_w;
  // modes 1 and 3: distance in elements between neighbouring pixels, rows and images of the
  // activation codes (0: dense NHWC, i.e. Cin, W * Cin, H * W * Cin)
  int64_t pix_pitch, row_pitch, img_pitch;
};

struct GemmArgs {
  const ConvArgs* conv;  // null for linear layers
  // D[Mr, Nc] = A * B over contraction length Kc.
  // a_mn = 0: A is stored [Mr, Kc] row-major; a_mn = 1: A is stored [Kc, Mr] row-major.
  // b_mn = 0: B is stored [Nc, Kc] row-major; b_mn = 1: B is stored [Kc, Nc] row-major.
  const bf16* A;
  const bf16* B;
  int64_t Mr, Nc, Kc;
  int64_t lda, ldb;  // row pitch in elements of the stored matrices
  int a_mn, b_mn;
  int epi;
  int out_bf16;      // EPI_FWD / EPI_DX: output dtype
  void* out;         // EPI_FWD: Y [Mr,Nc]; EPI_DX: dX [Mr,Nc]; EPI_PART: fp32 partials
  int64_t ldo;
  // EPI_FWD
  const float* col_scale;  // s_w[Nc]
  const float* col_bias;   // bias[Nc] or null
  // EPI_FWD with 8-bit integer operands (kind::i8, K-major, plain matrices): A = activation codes
  // (not centred), B = weight codes, wsum[n] = sum_k B[n,k]; the epilogue subtracts Zr * wsum[n]
  int i8; const int32_t* wsum;
  // EPI_FWD / EPI_DX: learnable activation scale / zero point and their bit-width
  const float* s_x; const float* z_x; int x_bits, x_sym;
  // EPI_DX
  const void* X;     // raw activations [Mr,Nc] in x_dtype
  int x_dtype;
  float* partials;   // [gemm_dx_num_partials][2]
  int64_t partials_cap;   // EPI_DX: pairs available at `partials` (0: not checked)
  // EPI_PART: out[split*split_stride + col*ldo + row], col < part_cols only
  int splits;
  int64_t split_stride;
  int64_t part_cols;
  int* status;
  // 1: this launch reads nothing that the launch directly before it in the stream writes, and
  // everything else it reads was complete before that launch began its work; it may then run
  // beside its predecessor (see gemm_kernel)
  int defer_wait;
};
// Tiled tensor map over a row-major matrix [rows, cols] with pitch ld (elements): box = row_bytes
// (128 or 64: the swizzle span) of columns x box_rows rows.  kind: 0 fp32, 1 bf16, 2 8-bit.
int tensor_map_2d(CUtensorMap* m, const void* base, int kind, int64_t rows, int64_t cols, int64_t ld, int box_rows,
                  int row_bytes);
// Number of (dS_x, dZ_x) partial pairs EPI_DX writes for this problem.
int gemm_dx_num_partials(int64_t Mr, int64_t Nc);
// Split count along the contraction for EPI_PART.
int gemm_choose_splits(int64_t Mr, int64_t Nc, int64_t Kc, int sm_count);
// Once per device with that device current: resolves the tensor-map encoder and lets every
// instantiation of the GEMM kernel use the full shared memory; returns an efqat_status.
int gemm_init();
void conv_pixel_box(int W, int H, int B, int target, int* tw, int* th, int* tb);
// tiles_out (optional): number of output tiles = number of partial pairs EPI_DX wrote.
// grid_out (optional): number of CTAs launched.
int run_gemm(const GemmArgs& a, int sm_count, cudaStream_t st, int* tiles_out = nullptr, int* grid_out = nullptr);
// Output tiles of an EPI_PART problem (before the split of the contraction).
int64_t gemm_part_tiles(int64_t Mr, int64_t Nc);

}  // namespace efqat
