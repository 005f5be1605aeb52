// C ABI of the library: argument validation, workspace carving and the launch sequence
// of each entry point.  Every step of the path runs in this library's kernels; there is
// no host fallback.
#include <new>
#include <vector>

#include "../../include/efqat_aux.h"
#include "internal.h"

using namespace efqat;

static const int PROF_KINDS = 3;       // 0 forward GEMM, 1 grad-input GEMM, 2 weight-grad GEMM
static const int PROF_RING = 8192;     // event pairs kept per kind between two reads

struct efqat_ctx {
  int device;
  int sm_count;
  int* d_status;
  long long launches;     // kernels launched through this context
  int prof_on;
  std::vector<cudaEvent_t> ev[PROF_KINDS];   // start/stop pairs, created by efqat_profile_enable
  int ev_used[PROF_KINDS];
};

// The context whose entry point is executing on this thread: launchers deep in the call tree
// add to its counter without every signature carrying the context.
static thread_local efqat_ctx* t_ctx = nullptr;
namespace efqat {
void count_launches(int n) {
  if (t_ctx) t_ctx->launches += n;
}
}  // namespace efqat
namespace {
struct Entered {
  explicit Entered(efqat_ctx* c) { t_ctx = c; }
  ~Entered() { t_ctx = nullptr; }
};
}  // namespace

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Output extent of a convolution along one axis.
inline int64_t conv_out(int64_t in, int64_t filt, int64_t pad, int64_t stride) {
  return (in + 2 * pad - filt) / stride + 1;
}

int check_bits(const efqat_qspec* q) {
  if (!q) return EFQAT_ERR_NULL;
  if (q->w_bits < 2 || q->w_bits > 8 || q->x_bits < 2 || q->x_bits > 8) return EFQAT_ERR_BITS;
  return EFQAT_OK;
}

int check_layer(const efqat_layer_desc* l, const efqat_qspec* q) {
  if (!l) return EFQAT_ERR_NULL;
  int rc = check_bits(q);
  if (rc != EFQAT_OK) return rc;
  if (l->act_dtype != EFQAT_F32 && l->act_dtype != EFQAT_BF16) return EFQAT_ERR_DTYPE;
  if (l->M < 1 || l->N < 1 || l->K < 1) return EFQAT_ERR_SHAPE;
  if (l->M > INT32_MAX || l->N > INT32_MAX || l->K > INT32_MAX) return EFQAT_ERR_SHAPE;
  if ((l->N & 7) || (l->K & 7)) return EFQAT_ERR_ALIGN;
  if (l->is_conv) {
    if (l->B < 1 || l->H < 1 || l->W < 1 || l->Cin < 1 || l->R < 1 || l->S < 1) return EFQAT_ERR_SHAPE;
    if (l->stride < 1) return EFQAT_ERR_SHAPE;
    if (l->stride > 2 || l->R * l->S > 49) return EFQAT_ERR_UNIMPL;     // strides 1 and 2, filters up to 7 x 7
    if (l->pad < 0 || l->pad >= l->R || l->pad >= l->S) return EFQAT_ERR_SHAPE;
    if (l->Cin & 7) return EFQAT_ERR_ALIGN;
    if (l->H + 2 * l->pad < l->R || l->W + 2 * l->pad < l->S) return EFQAT_ERR_SHAPE;
    const int64_t Ho = conv_out(l->H, l->R, l->pad, l->stride), Wo = conv_out(l->W, l->S, l->pad, l->stride);
    if (l->M != static_cast<int64_t>(l->B) * Ho * Wo) return EFQAT_ERR_SHAPE;
    if (l->K != static_cast<int64_t>(l->R) * l->S * l->Cin) return EFQAT_ERR_SHAPE;
  }
  return EFQAT_OK;
}

// Workspace sections of the forward / backward calls.
struct LayerWs {
  ActQ* actq;
  bf16* Xc;        // [M,K] centred activation codes
  bf16* Wq;        // [N,K] weight codes (forward) or dequantised weights (backward)
  bf16* dYb;       // [M,N] bf16 copy of an fp32 dY
  bf16* dYsel;     // [M,pitch] gathered selected columns of dY
  float* P;        // [splits][k_sel][K] partial weight-gradient products
  float* dxpart;   // [tiles][2]
  float* colsum;   // [COLSUM_SLABS][N]
  int32_t* wsum;   // [N] row sums of the 8-bit weight codes (integer forward)
  bf16* strip;     // [N, R * nP * 64] banded weights of the strip-form grad-input (few input channels)
  int64_t pitch;
  int splits;
  size_t bytes;
};

int64_t sel_pitch(int64_t k_sel) { return round_up(k_sel, 64); }

// A 1x1 convolution with stride 1 and no padding is the linear layer on the [B*H*W, Cin] matrix.
bool spatial_conv(const efqat_layer_desc* l) {
  return l->is_conv && (l->R != 1 || l->S != 1 || l->pad != 0 || l->stride != 1);
}

ConvArgs conv_args(const efqat_layer_desc* l, int mode) {
  ConvArgs c = {};
  c.mode = mode;
  c.B = l->B; c.H = l->H; c.W = l->W; c.Cin = l->Cin;
  c.Ho = static_cast<int>(conv_out(l->H, l->R, l->pad, l->stride));
  c.Wo = static_cast<int>(conv_out(l->W, l->S, l->pad, l->stride));
  c.N = static_cast<int>(l->N);
  c.R = l->R; c.S = l->S; c.pad = l->pad;
  c.stride = l->stride;
  return c;
}

int64_t x_elems(const efqat_layer_desc* l) {
  return spatial_conv(l) ? static_cast<int64_t>(l->B) * l->H * l->W * l->Cin : l->M * l->K;
}

// Convolutions with few input channels (the 7 x 7 input layer on 8 stored channels): one filter
// row covers S * Cin <= 64 contiguous elements of an NHWC image row, so a whole filter row is one
// 64-wide contraction block instead of S blocks that are mostly zero fill.  The forward and the
// weight-gradient GEMMs then see an R x 1 convolution with S * Cin "channels" on a virtual image
// whose pixel w starts at stored pixel w (pixels overlap: the pixel pitch stays Cin elements).
// The horizontal padding cannot come from TMA's out-of-range fill in this view, so the
// activation codes are written into a zero-framed image [B, H + 2 pad, W + 2 pad, Cin].
bool narrow_conv(const efqat_layer_desc* l) {
  return spatial_conv(l) && l->S > 1 && l->S * l->Cin <= 64;
}

ConvArgs conv_args_x(const efqat_layer_desc* l, int mode) {
  ConvArgs c = conv_args(l, mode);
  if (!narrow_conv(l)) return c;
  const int64_t Hp = l->H + 2 * l->pad, Wp = l->W + 2 * l->pad;
  c.H = static_cast<int>(Hp);
  c.W = (c.Wo - 1) * l->stride + 1;          // virtual pixels 0, stride, ... are the first taps of the outputs
  c.Cin = l->S * l->Cin;
  c.S = 1;
  c.pad = 0;
  c.pix_pitch = l->Cin;
  c.row_pitch = Wp * l->Cin;
  c.img_pitch = Hp * Wp * l->Cin;
  return c;
}

// elements of the activation-code buffer
int64_t xc_elems(const efqat_layer_desc* l) {
  if (!narrow_conv(l)) return x_elems(l);
  return static_cast<int64_t>(l->B) * (l->H + 2 * l->pad) * (l->W + 2 * l->pad) * l->Cin;
}

// Strip form of the grad-input of such a layer.  With Cin stored channels, P = 64 / Cin input pixels
// of one image row are 64 contiguous elements of dX: they become ONE output row of the GEMM (64
// columns instead of Cin), fed by the nP output columns that reach the strip, through a banded
// copy of the weights (StripArgs).  One launch per class of input ROWS (stride classes); along W
// the stride is absorbed by the band.  dY is read through up to four views whose pixel pitch is
// Q = P / stride output pixels (one per residue of the output column modulo Q).
struct StripGeo {
  bool ok;
  int P, Q, p_min, nP;
};

StripGeo strip_geo(const efqat_layer_desc* l) {
  StripGeo g = {};
  if (!narrow_conv(l) || 64 % l->Cin != 0) return g;
  g.P = 64 / l->Cin;
  if (l->W % g.P != 0 || g.P % l->stride != 0) return g;
  g.Q = g.P / l->stride;
  if (g.Q > 4) return g;
  const int lo = l->pad - (l->S - 1);                       // smallest stride * p that still reaches pixel q = 0
  g.p_min = lo >= 0 ? (lo + l->stride - 1) / l->stride : -((-lo) / l->stride);
  const int p_max = (g.P - 1 + l->pad) / l->stride;
  g.nP = p_max - g.p_min + 1;
  if (g.nP < 1 || (l->R + l->stride - 1) / l->stride * g.nP > 49 || l->R * g.nP > 255) return g;
  g.ok = true;
  return g;
}

void set_x_layout(PrepArgs* pa, const efqat_layer_desc* l) {
  if (!narrow_conv(l)) return;
  pa->xp_C8 = l->Cin / 8; pa->xp_H = l->H; pa->xp_W = l->W; pa->xp_pad = l->pad;
}

// (dS_x, dZ_x) partial pairs of the grad-input launches: for a convolution, one launch per class
// of input pixels (stride x stride classes), each tiled by its own pixel box.
// Upper bound of the 128-pixel boxes a grad-input launch may cut a W x H x B pixel space into: the
// least-waste box, or one of the one-image boxes of a launch whose taps share boxes per filter column.
int64_t dx_boxes(int64_t Wc, int64_t Hc, int64_t Bn) {
  int tw, th, tb;
  conv_pixel_box(static_cast<int>(Wc), static_cast<int>(Hc), static_cast<int>(Bn), 128, &tw, &th, &tb);
  int64_t boxes = ceil_div(Wc, tw) * ceil_div(Hc, th) * ceil_div(Bn, tb);
  const int cand[2][2] = {{8, 16}, {16, 8}};
  for (int i = 0; i < 2; ++i) {
    const int64_t b2 = ceil_div(Wc, cand[i][0]) * ceil_div(Hc, cand[i][1]) * Bn;
    if (b2 * 128 <= (23 * Wc * Hc * Bn) / 20 + 128 && b2 > boxes) boxes = b2;
  }
  return boxes;
}

int dx_partials(const efqat_layer_desc* l) {
  if (!spatial_conv(l)) return gemm_dx_num_partials(l->M, l->K);
  int64_t n = 0;
  const StripGeo sg = strip_geo(l);
  for (int ah = 0; ah < l->stride; ++ah) {
    const int64_t Hc = ceil_div(l->H - ah, l->stride);
    if (Hc < 1) continue;
    if (sg.ok) {                      // strips of P pixels: one launch per class of input rows, 64 columns
      n += dx_boxes(l->W / sg.P, Hc, l->B) * 8;
      continue;
    }
    for (int aw = 0; aw < l->stride; ++aw) {
      const int64_t Wc = ceil_div(l->W - aw, l->stride);
      if (Wc < 1) continue;
      n += dx_boxes(Wc, Hc, l->B) * ceil_div(l->Cin, 64) * 8;
    }
  }
  return static_cast<int>(n);
}

// Layers whose backward runs in one pass over dY and X (skinny_bwd.cu).
bool one_pass_bwd(const efqat_layer_desc* l) {
  return !spatial_conv(l) && skinny_bwd_applies(l->M, l->N, l->K, l->act_dtype == EFQAT_BF16);
}

LayerWs carve(void* ws, const efqat_layer_desc* l, int64_t k_sel, int sm_count, int64_t p_elems_override) {
  LayerWs w = {};
  char* base = ws ? reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~uintptr_t(255)) : nullptr;
  size_t off = 0;
  auto take = [&](int64_t bytes) {
    char* r = base ? base + off : nullptr;
    off += static_cast<size_t>(round_up(bytes, 256));
    return r;
  };
  const int64_t M = l->M, N = l->N, K = l->K;
  w.actq = reinterpret_cast<ActQ*>(take(sizeof(ActQ)));
  w.Xc = reinterpret_cast<bf16*>(take(xc_elems(l) * 2));
  w.Wq = reinterpret_cast<bf16*>(take(N * K * 2));
  w.dYb = reinterpret_cast<bf16*>(take(l->act_dtype == EFQAT_F32 ? M * N * 2 : 0));
  const bool gathered = k_sel > 0 && k_sel < N;
  w.pitch = gathered ? sel_pitch(k_sel) : N;
  w.dYsel = reinterpret_cast<bf16*>(take(gathered ? M * w.pitch * 2 : 0));
  w.splits = k_sel > 0 ? gemm_choose_splits(K, gathered ? round_up(k_sel, 16) : N, M, sm_count) : 1;
  if (k_sel > 0 && one_pass_bwd(l)) w.splits = skinny_bwd_grid(M, sm_count);     // one partial product per CTA
  const int64_t p_elems = p_elems_override >= 0 ? p_elems_override : static_cast<int64_t>(w.splits) * k_sel * K;
  w.P = reinterpret_cast<float*>(take(p_elems * 4));
  w.dxpart = reinterpret_cast<float*>(take(static_cast<int64_t>(dx_partials(l)) * 8));
  w.colsum = reinterpret_cast<float*>(take(static_cast<int64_t>(prepare_slabs(M, N)) * N * 4));
  w.wsum = reinterpret_cast<int32_t*>(take(N * 4));
  const StripGeo sg = strip_geo(l);
  w.strip = reinterpret_cast<bf16*>(take(sg.ok ? N * l->R * sg.nP * 64 * 2 : 0));
  w.bytes = off + 256;
  return w;
}

// A plain layer runs its forward on the integer tensor cores: 8-bit codes, int32 accumulation,
// zero point taken out exactly in the epilogue.  int32 holds K * 255 * 127 up to K = 65536; the
// limit here leaves a factor 2.  The row pitch of the 8-bit operands must be a multiple of 16
// bytes for TMA, and tiles are kept to multiples of 32 columns, the coarser of the instruction's
// N granularities.  Short contractions (K <= 256: output-bound layers whose 128-wide k-blocks
// would be half padding) measured slower this way and stay on the bf16 path.
bool fwd_on_i8(const efqat_layer_desc* l) {
  return !spatial_conv(l) && l->K >= 512 && l->K <= 32768 && l->K % 16 == 0 && l->N % 32 == 0;
}

// Sections of a layer's weight-operand cache (see cache.cu).
struct WCache {
  int8_t* codes8;     // [N,K] 8-bit codes (integer forward) ...
  int32_t* wsum;      // [N] ... and their row sums
  bf16* codes16;      // [N,K] codes as bf16 (every other forward)
  bf16* what;         // [N,K] dequantised weights (grad-input GEMM)
  size_t bytes;
};

WCache carve_cache(void* cache, const efqat_layer_desc* l) {
  WCache c = {};
  char* base = cache ? reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(cache) + 255) & ~uintptr_t(255)) : nullptr;
  size_t off = 0;
  auto take = [&](int64_t bytes) {
    char* r = base ? base + off : nullptr;
    off += static_cast<size_t>(round_up(bytes, 256));
    return r;
  };
  const int64_t nk = l->N * l->K;
  if (fwd_on_i8(l)) {
    c.codes8 = reinterpret_cast<int8_t*>(take(nk));
    c.wsum = reinterpret_cast<int32_t*>(take(l->N * 4));
  } else {
    c.codes16 = reinterpret_cast<bf16*>(take(nk * 2));
  }
  c.what = reinterpret_cast<bf16*>(take(nk * 2));
  c.bytes = off + 256;
  return c;
}

int guard_device(const efqat_ctx* ctx) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != ctx->device) return EFQAT_ERR_CUDA;
  return EFQAT_OK;
}

int last_error() { return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA; }

// run_gemm, bracketed by a pair of events when per-kernel timing is switched on.
int timed_gemm(efqat_ctx* ctx, int kind, const GemmArgs& g, cudaStream_t st, int* tiles = nullptr,
               int* grid = nullptr) {
  const bool rec = ctx->prof_on && ctx->ev_used[kind] < PROF_RING;
  const int slot = ctx->ev_used[kind];
  if (rec) cudaEventRecord(ctx->ev[kind][2 * slot], st);
  const int rc = run_gemm(g, ctx->sm_count, st, tiles, grid);
  if (rec) {
    cudaEventRecord(ctx->ev[kind][2 * slot + 1], st);
    ctx->ev_used[kind] = slot + 1;
  }
  return rc;
}

}  // namespace

extern "C" {

int efqat_create(efqat_ctx** out, int device) {
  if (!out) return EFQAT_ERR_NULL;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return EFQAT_ERR_CUDA;
  int prev = 0;
  cudaGetDevice(&prev);
  if (cudaSetDevice(device) != cudaSuccess) return EFQAT_ERR_CUDA;
  efqat_ctx* c = new (std::nothrow) efqat_ctx();
  if (!c) return EFQAT_ERR_CUDA;
  c->device = device;
  c->prof_on = 0;
  c->launches = 0;
  for (int k = 0; k < PROF_KINDS; ++k) c->ev_used[k] = 0;
  int rc = EFQAT_OK;
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
      cudaMalloc(&c->d_status, 256) != cudaSuccess || cudaMemset(c->d_status, 0, 256) != cudaSuccess)
    rc = EFQAT_ERR_CUDA;
  if (rc == EFQAT_OK) rc = gemm_init();
  cudaSetDevice(prev);
  if (rc != EFQAT_OK) {
    delete c;
    return rc;
  }
  *out = c;
  return EFQAT_OK;
}

int efqat_destroy(efqat_ctx* ctx) {
  if (!ctx) return EFQAT_ERR_NULL;
  if (ctx->d_status) cudaFree(ctx->d_status);
  for (int k = 0; k < PROF_KINDS; ++k)
    for (cudaEvent_t e : ctx->ev[k]) cudaEventDestroy(e);
  delete ctx;
  return EFQAT_OK;
}

const char* efqat_status_string(int s) {
  switch (s) {
    case EFQAT_OK: return "ok";
    case EFQAT_ERR_NULL: return "required pointer is NULL";
    case EFQAT_ERR_SHAPE: return "invalid or inconsistent shape";
    case EFQAT_ERR_ALIGN: return "alignment contract violated";
    case EFQAT_ERR_DTYPE: return "unknown dtype";
    case EFQAT_ERR_BITS: return "bit-width outside [2,8]";
    case EFQAT_ERR_MODE: return "unknown selection mode";
    case EFQAT_ERR_WORKSPACE: return "workspace missing or too small";
    case EFQAT_ERR_K_RANGE: return "selection count out of range";
    case EFQAT_ERR_UNIMPL: return "combination not implemented";
    case EFQAT_ERR_CUDA: return "CUDA call failed";
    case EFQAT_ERR_TOO_LARGE: return "size exceeds a built-in maximum";
    case EFQAT_DEV_BAD_SCALE: return "device: scale not positive and finite";
    case EFQAT_DEV_BAD_INDEX: return "device: channel index out of range or not ascending";
    case EFQAT_DEV_WAIT_TIMEOUT: return "device: bounded wait expired";
    default: return "unknown status";
  }
}

int efqat_device_status(efqat_ctx* ctx, int* code) {
  if (!ctx || !code) return EFQAT_ERR_NULL;
  const int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  if (cudaDeviceSynchronize() != cudaSuccess) return EFQAT_ERR_CUDA;
  if (cudaMemcpy(code, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return EFQAT_ERR_CUDA;
  if (cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess) return EFQAT_ERR_CUDA;
  return EFQAT_OK;
}

int efqat_profile_enable(efqat_ctx* ctx, int enable) {
  if (!ctx) return EFQAT_ERR_NULL;
  int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  if (enable && ctx->ev[0].empty()) {
    for (int k = 0; k < PROF_KINDS; ++k) {
      ctx->ev[k].resize(2 * PROF_RING);
      for (auto& e : ctx->ev[k])
        if (cudaEventCreate(&e) != cudaSuccess) return EFQAT_ERR_CUDA;
    }
  }
  for (int k = 0; k < PROF_KINDS; ++k) ctx->ev_used[k] = 0;
  ctx->prof_on = enable ? 1 : 0;
  return EFQAT_OK;
}

int efqat_profile_read(efqat_ctx* ctx, int which, float* ms_total, int* launches) {
  if (!ctx || !ms_total || !launches) return EFQAT_ERR_NULL;
  if (which < 0 || which >= PROF_KINDS) return EFQAT_ERR_MODE;
  const int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  if (cudaDeviceSynchronize() != cudaSuccess) return EFQAT_ERR_CUDA;
  double total = 0.0;
  for (int i = 0; i < ctx->ev_used[which]; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev[which][2 * i], ctx->ev[which][2 * i + 1]) != cudaSuccess)
      return EFQAT_ERR_CUDA;
    total += ms;
  }
  *ms_total = static_cast<float>(total);
  *launches = ctx->ev_used[which];
  ctx->ev_used[which] = 0;
  return EFQAT_OK;
}

int64_t efqat_launch_count(efqat_ctx* ctx) { return ctx ? static_cast<int64_t>(ctx->launches) : 0; }

int efqat_selftest_bounded_wait(efqat_ctx* ctx, uint64_t limit_ns, efqat_stream_t stream) {
  if (!ctx) return EFQAT_ERR_NULL;
  if (limit_ns < 1000 || limit_ns > 1000000000ull) return EFQAT_ERR_SHAPE;    // 1 us .. 1 s
  const int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_wait_selftest(ctx->d_status, limit_ns, stream);
  return last_error();
}

int64_t efqat_ratio_to_k(double ratio, int64_t n) {
  if (!(ratio > 0.0) || n <= 0) return 0;
  if (ratio >= 1.0) return n;
  return static_cast<int64_t>(floor(ratio * static_cast<double>(n)));
}

int efqat_validate_layer(const efqat_layer_desc* layer, const efqat_qspec* q) { return check_layer(layer, q); }

int efqat_workspace_bytes(const efqat_layer_desc* layer, const efqat_qspec* q, int64_t k_sel_max, size_t* out) {
  if (!out) return EFQAT_ERR_NULL;
  int rc = check_layer(layer, q);
  if (rc != EFQAT_OK) return rc;
  if (k_sel_max < 0 || k_sel_max > layer->N) return EFQAT_ERR_K_RANGE;
  // the partial-product buffer is the only section that is not monotone in k_sel
  // (fewer channels -> more splits of the contraction); take its maximum.  The split rule
  // depends on the SM count: that of the current CUDA device, the one the compute calls
  // require to be current as well (148, a B200, where no device can be asked).
  int sm = 148, dev = -1, n = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 &&
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
    sm = n;
  else
    cudaGetLastError();
  int64_t p_max = 0;
  for (int64_t k = 1; k <= k_sel_max; ++k) {
    const int64_t nc = (k < layer->N) ? round_up(k, 16) : layer->N;
    const int64_t sp = one_pass_bwd(layer) ? skinny_bwd_grid(layer->M, sm) : gemm_choose_splits(layer->K, nc, layer->M, sm);
    const int64_t e = sp * k * layer->K;
    if (e > p_max) p_max = e;
  }
  // dYsel is largest for the largest gathered k
  const int64_t k_g = (k_sel_max == layer->N && layer->N > 1) ? layer->N - 1 : k_sel_max;
  *out = carve(nullptr, layer, k_g, sm, p_max).bytes;
  return EFQAT_OK;
}

int efqat_select_workspace_bytes(int L, int64_t total_channels, size_t* out) {
  if (!out) return EFQAT_ERR_NULL;
  if (L < 1 || total_channels < 1) return EFQAT_ERR_SHAPE;
  *out = select_workspace_bytes(L, total_channels) + 256;
  return EFQAT_OK;
}

int efqat_select_channels(efqat_ctx* ctx, int mode, int L, const efqat_layer_desc* layers,
                          const float* const* weights, const int64_t* k, int32_t* idx, int32_t* offsets,
                          float* importance_or_null, void* ws, size_t ws_bytes, efqat_stream_t stream) {
  if (!ctx || !layers || !weights || !k || !offsets) return EFQAT_ERR_NULL;
  if (L < 1) return EFQAT_ERR_SHAPE;
  if (mode != EFQAT_CWPL && mode != EFQAT_CWPN && mode != EFQAT_LWPN) return EFQAT_ERR_MODE;
  if (!ws) return EFQAT_ERR_WORKSPACE;
  int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  void* base = reinterpret_cast<void*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~uintptr_t(255));
  const size_t slack = static_cast<size_t>(reinterpret_cast<char*>(base) - reinterpret_cast<char*>(ws));
  if (ws_bytes < slack) return EFQAT_ERR_WORKSPACE;
  if (!idx) {
    // idx may only be NULL when nothing can be selected
    int64_t want = 0;
    for (int l = 0; l < (mode == EFQAT_CWPL ? L : 1); ++l) want += k[l];
    if (want > 0) return EFQAT_ERR_NULL;
  }
  Entered in(ctx);
  return run_select(mode, L, layers, weights, k, idx, offsets, importance_or_null, base, ws_bytes - slack,
                    ctx->d_status, stream);
}

}  // extern "C"

namespace {

// Forward of one layer.  cache != NULL: the weight operand comes from the layer's cache and W is
// not read (it may be NULL).
int fwd_impl(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* X, const float* W,
             const float* s_w, const float* s_x, const float* z_x, const float* bias_or_null, void* Y, void* ws,
             size_t ws_bytes, const void* cache, size_t cache_bytes, efqat_stream_t stream) {
  if (!ctx || !X || (!W && !cache) || !s_w || !s_x || !Y) return EFQAT_ERR_NULL;
  int rc = check_layer(layer, q);
  if (rc != EFQAT_OK) return rc;
  if (!q->x_symmetric && !z_x) return EFQAT_ERR_NULL;
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y)) return EFQAT_ERR_ALIGN;
  if (!ws) return EFQAT_ERR_WORKSPACE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  const LayerWs w = carve(ws, layer, 0, ctx->sm_count, 0);
  if (ws_bytes < w.bytes) return EFQAT_ERR_WORKSPACE;
  WCache wc = {};
  if (cache) {
    wc = carve_cache(const_cast<void*>(cache), layer);
    if (cache_bytes < wc.bytes) return EFQAT_ERR_WORKSPACE;
  }
  Entered in(ctx);
  const int64_t M = layer->M, N = layer->N, K = layer->K;
  cudaStream_t st = stream;

  const int act_bf16 = layer->act_dtype == EFQAT_BF16;
  // short contractions (HBM-bound layers): one launch, X and Y touched once
  if (!spatial_conv(layer) && skinny_fwd_applies(M, N, K, act_bf16)) {
    rc = run_skinny_fwd(M, N, K, act_bf16, X, Y, W, cache ? wc.codes16 : nullptr, s_w, s_x, z_x, bias_or_null,
                        q->w_bits, q->x_bits, q->x_symmetric, ctx->d_status, ctx->sm_count, st);
    return rc != EFQAT_OK ? rc : last_error();
  }
  // a2: both quantizers in one launch
  PrepArgs pa = {};
  pa.M = M; pa.N = N; pa.K = K;
  pa.W = cache ? nullptr : W; pa.s_w = s_w; pa.w_bits = q->w_bits; pa.Wq = w.Wq;
  pa.X = X; pa.s_x = s_x; pa.z_x = z_x; pa.x_bits = q->x_bits; pa.x_sym = q->x_symmetric; pa.Xc = w.Xc;
  pa.x_count = x_elems(layer);
  set_x_layout(&pa, layer);
  pa.status = ctx->d_status;
  // integer forward: the code buffers of the bf16 path are reused, half filled
  const bool i8 = fwd_on_i8(layer);
  if (i8) {
    pa.i8 = 1;
    pa.Wq8 = reinterpret_cast<int8_t*>(w.Wq);
    pa.Xc8 = reinterpret_cast<uint8_t*>(w.Xc);
    pa.wsum = w.wsum;
  }
  launch_prepare(pa, 0, act_bf16, st);
  ConvArgs cva;
  GemmArgs g = {};
  g.i8 = i8 ? 1 : 0;
  g.wsum = cache ? wc.wsum : w.wsum;
  g.A = w.Xc;
  g.B = !cache ? w.Wq : (i8 ? reinterpret_cast<const bf16*>(wc.codes8) : wc.codes16);
  g.Mr = M; g.Nc = N; g.Kc = K;
  g.lda = K; g.ldb = K;
  g.a_mn = 0; g.b_mn = 0;
  g.epi = EPI_FWD;
  g.out_bf16 = layer->act_dtype == EFQAT_BF16;
  g.out = Y; g.ldo = N;
  g.col_scale = s_w; g.col_bias = bias_or_null;
  g.s_x = s_x; g.z_x = z_x; g.x_bits = q->x_bits; g.x_sym = q->x_symmetric;
  if (spatial_conv(layer)) {
    cva = conv_args_x(layer, 1);
    g.conv = &cva;
  }
  g.status = ctx->d_status;
  rc = timed_gemm(ctx, 0, g, st);
  if (rc != EFQAT_OK) return rc;
  return last_error();
}

// Backward of one layer.  cache != NULL: the grad-input GEMM reads the dequantised weights of the
// layer's cache instead of rebuilding them (W is still read for the clip mask of the unfrozen rows).
// Chaining of the finalize launches over the layers of a network backward: a layer's finalize work
// (reduction of its partial products, clip masks, dS / db, optional SGD) is independent of the next
// layer's prepare jobs, so it may ride in that layer's prepare launch instead of a launch of its own.
struct FinChain {
  FinArgs pending;       // finalize work of the layer before, not launched yet
  bool has_pending;
  bool defer;            // this layer's finalize may be left pending for the next call
};

// Only light finalize work is worth carrying: one block per unfrozen row reads that row of every split
// partial product, and with many rows behind another layer's prepare jobs it only delays the GEMMs that
// wait for that launch (measured on the 144-layer stack, everything carried: 100 % backward 18.0 ->
// 19.6 ms while 10 % went 12.1 -> 11.5 ms).
bool fin_is_light(const FinArgs& f) { return f.k_sel <= 512; }

int bwd_impl(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* dY, const void* X,
             const float* W, const float* s_w, const float* s_x, const float* z_x, const int32_t* idx, int64_t k_sel,
             void* dX, float* dW_sel, float* dS_w_sel, float* dS_x, float* dZ_x, float* db_or_null,
             const efqat_sgd* opt_or_null, void* ws, size_t ws_bytes, const void* cache, size_t cache_bytes,
             efqat_stream_t stream, FinChain* chain = nullptr) {
  if (!ctx || !dY || !X || !W || !s_w || !s_x || !dX || !dS_x || !dZ_x) return EFQAT_ERR_NULL;
  int rc = check_layer(layer, q);
  if (rc != EFQAT_OK) return rc;
  if (!q->x_symmetric && !z_x) return EFQAT_ERR_NULL;
  const int64_t M = layer->M, N = layer->N, K = layer->K;
  if (k_sel < 0 || k_sel > N) return EFQAT_ERR_K_RANGE;
  if (k_sel > 0 && (!dW_sel || !dS_w_sel)) return EFQAT_ERR_NULL;
  if (k_sel > 0 && k_sel < N && !idx) return EFQAT_ERR_NULL;
  if (opt_or_null && k_sel > 0 && (!opt_or_null->W_inout || !opt_or_null->mom_inout)) return EFQAT_ERR_NULL;
  if (opt_or_null && k_sel > 0 && (!aligned16(opt_or_null->W_inout) || !aligned16(opt_or_null->mom_inout)))
    return EFQAT_ERR_ALIGN;
  if (dS_w_sel == nullptr && k_sel > 0) return EFQAT_ERR_NULL;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(W) || !aligned16(dX) || (dW_sel && !aligned16(dW_sel)))
    return EFQAT_ERR_ALIGN;
  if (!ws) return EFQAT_ERR_WORKSPACE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  const LayerWs w = carve(ws, layer, k_sel, ctx->sm_count, -1);
  if (ws_bytes < w.bytes) return EFQAT_ERR_WORKSPACE;
  WCache wc = {};
  if (cache) {
    wc = carve_cache(const_cast<void*>(cache), layer);
    if (cache_bytes < wc.bytes) return EFQAT_ERR_WORKSPACE;
  }
  Entered in(ctx);
  cudaStream_t st = stream;
  const int act_bf16 = layer->act_dtype == EFQAT_BF16;

  const bool gathered = k_sel > 0 && k_sel < N;
  if (one_pass_bwd(layer)) {
    // short contraction: one launch reads dY and X once and leaves per-CTA partials for the finalize launch
    const int grid = skinny_bwd_grid(M, ctx->sm_count);
    if (chain && chain->has_pending) {          // no prepare launch here to carry it
      launch_finalize(chain->pending, st);
      chain->has_pending = false;
    }
    rc = run_skinny_bwd(M, N, dY, X, dX, W, cache ? wc.what : nullptr, s_w, q->w_bits, s_x, z_x, q->x_bits,
                        q->x_symmetric, gathered ? idx : nullptr, k_sel, w.P, db_or_null ? w.colsum : nullptr, w.dxpart,
                        ctx->d_status, ctx->sm_count, st);
    if (rc != EFQAT_OK) return rc;
    FinArgs fa = {};
    fa.N = N; fa.K = K; fa.k_sel = k_sel;
    fa.P = w.P; fa.splits = grid; fa.split_stride = k_sel * K;
    fa.W = W; fa.s_w = s_w; fa.s_x = s_x; fa.w_bits = q->w_bits;
    fa.idx = gathered ? idx : nullptr;
    fa.dW_sel = dW_sel; fa.dS_w_sel = dS_w_sel;
    if (opt_or_null) fa.opt = *opt_or_null;
    fa.has_opt = opt_or_null != nullptr;
    fa.dx_partials = w.dxpart; fa.n_partials = grid * 8; fa.dS_x = dS_x; fa.dZ_x = dZ_x;
    fa.colsum_ws = w.colsum; fa.slabs = grid; fa.db = db_or_null;
    fa.status = ctx->d_status;
    if (chain && chain->defer && fin_is_light(fa)) {
      chain->pending = fa;
      chain->has_pending = true;
    } else {
      launch_finalize(fa, st);
    }
    return last_error();
  }
  // a2: one launch: dequantised weight operand, activation codes (only when some channel is
  // unfrozen) and one pass over dY (column-sum partials, gathered columns, bf16 copy)
  const bf16* dYb = act_bf16 ? static_cast<const bf16*>(dY) : w.dYb;
  PrepArgs pa = {};
  pa.M = M; pa.N = N; pa.K = K;
  pa.W = cache ? nullptr : W; pa.s_w = s_w; pa.w_bits = q->w_bits; pa.Wq = w.Wq;
  pa.X = X; pa.s_x = s_x; pa.z_x = z_x; pa.x_bits = q->x_bits; pa.x_sym = q->x_symmetric;
  pa.Xc = k_sel > 0 ? w.Xc : nullptr;
  pa.x_count = x_elems(layer);
  set_x_layout(&pa, layer);
  pa.dY = dY; pa.dYb = act_bf16 ? nullptr : w.dYb;
  pa.colsum_ws = db_or_null ? w.colsum : nullptr;
  pa.idx = idx; pa.k_sel = k_sel; pa.pitch = w.pitch; pa.dYsel = gathered ? w.dYsel : nullptr;
  pa.status = ctx->d_status;
  launch_prepare(pa, 1, act_bf16, st, (chain && chain->has_pending) ? &chain->pending : nullptr);
  if (chain) chain->has_pending = false;
  // a4 + a5: dX = (dY W^) masked, with the dS_x / dZ_x partial sums in the epilogue
  int tiles = 0, dx_grid = 0, dw_splits = w.splits;
  const bool sconv = spatial_conv(layer);
  ConvArgs cv_dx = conv_args(layer, 2), cv_dw = conv_args_x(layer, 3);
  {
    GemmArgs g = {};
    if (sconv) g.conv = &cv_dx;
    g.A = dYb; g.B = cache ? wc.what : w.Wq;
    g.Mr = sconv ? x_elems(layer) / layer->Cin : M;
    g.Nc = sconv ? layer->Cin : K;
    g.Kc = sconv ? static_cast<int64_t>(layer->R) * layer->S * N : N;
    g.lda = N; g.ldb = K;
    g.a_mn = 0; g.b_mn = 1;
    g.epi = EPI_DX;
    g.out_bf16 = act_bf16;
    g.out = dX; g.ldo = sconv ? layer->Cin : K;
    g.s_x = s_x; g.z_x = z_x; g.x_bits = q->x_bits; g.x_sym = q->x_symmetric;
    g.X = X; g.x_dtype = layer->act_dtype;
    g.partials = w.dxpart;
    g.partials_cap = dx_partials(layer);
    g.status = ctx->d_status;
    if (!sconv) {
      rc = timed_gemm(ctx, 1, g, st, &tiles, &dx_grid);
      if (rc != EFQAT_OK) return rc;
    } else if (strip_geo(layer).ok) {
      // few input channels: strips of P pixels as GEMM rows, one launch per class of input rows
      const StripGeo sg = strip_geo(layer);
      StripArgs sa = {};
      sa.what = cache ? wc.what : w.Wq; sa.T = w.strip; sa.N = N;
      sa.R = layer->R; sa.S = layer->S; sa.Cin = layer->Cin; sa.pad = layer->pad; sa.stride = layer->stride;
      sa.p_min = sg.p_min; sa.nP = sg.nP;
      launch_strip_weights(sa, st);
      const int es = act_bf16 ? 2 : 4;
      const int64_t Ho = cv_dx.Ho, Wo = cv_dx.Wo, Cin = layer->Cin, Wd = layer->W, Hd = layer->H;
      g.B = w.strip;
      g.Nc = 64;
      g.Kc = static_cast<int64_t>(layer->R) * sg.nP * N;
      g.ldo = 64;
      for (int ah = 0; ah < layer->stride; ++ah) {
        const int64_t Hc = ceil_div(Hd - ah, static_cast<int64_t>(layer->stride));
        if (Hc < 1) continue;
        ConvExplicit ex = {};
        ex.pW = static_cast<int>(Wd / sg.P);
        ex.pH = static_cast<int>(Hc);
        for (int r = 0; r < layer->R; ++r) {
          const int nh = ah + layer->pad - r;
          if (nh % layer->stride != 0) continue;
          for (int pi = 0; pi < sg.nP; ++pi) {
            const int p = sg.p_min + pi;
            const int dwv = p >= 0 ? p / sg.Q : -((-p + sg.Q - 1) / sg.Q);     // floor(p / Q)
            const int t = ex.ntaps++;
            ex.tap_dh[t] = static_cast<int8_t>(nh / layer->stride);
            ex.tap_dw[t] = static_cast<int8_t>(dwv);
            ex.tap_map[t] = static_cast<uint8_t>(p - dwv * sg.Q);
            ex.tap_rs[t] = static_cast<uint8_t>(r * sg.nP + pi);
          }
        }
        for (int pm = 0; pm < sg.Q; ++pm) {
          ConvView& v = ex.a_view[pm];
          v.base = reinterpret_cast<const char*>(dYb) + static_cast<int64_t>(pm) * N * 2;
          v.W = Wo > pm ? ceil_div(Wo - pm, static_cast<int64_t>(sg.Q)) : 1;
          v.H = Ho;
          v.pix = static_cast<int64_t>(sg.Q) * N; v.row = Wo * N; v.img = Ho * Wo * N;
        }
        ex.o_view.base = static_cast<char*>(dX) + static_cast<int64_t>(ah) * Wd * Cin * es;
        ex.x_base = static_cast<const char*>(X) + static_cast<int64_t>(ah) * Wd * Cin * es;
        ex.o_view.W = Wd / sg.P; ex.o_view.H = Hc;
        ex.o_view.pix = 64; ex.o_view.row = static_cast<int64_t>(layer->stride) * Wd * Cin; ex.o_view.img = Hd * Wd * Cin;
        ex.b_cols = static_cast<int64_t>(layer->R) * sg.nP * 64;
        cv_dx.ex = &ex;
        if (ex.ntaps == 0) {
          // no filter row reaches this class of input rows: its gradient is zero
          for (int b = 0; b < layer->B; ++b)
            if (cudaMemset2DAsync(static_cast<char*>(dX) + (static_cast<int64_t>(b) * Hd + ah) * Wd * Cin * es,
                                  static_cast<size_t>(layer->stride) * Wd * Cin * es, 0,
                                  static_cast<size_t>(Wd) * Cin * es, static_cast<size_t>(Hc), st) != cudaSuccess)
              return EFQAT_ERR_CUDA;
          continue;
        }
        g.Mr = static_cast<int64_t>(layer->B) * Hc * (Wd / sg.P);
        g.partials = w.dxpart + 2 * static_cast<int64_t>(tiles);
        g.partials_cap = dx_partials(layer) - tiles;
        int t1 = 0, g1 = 0;
        rc = timed_gemm(ctx, 1, g, st, &t1, &g1);
        cv_dx.ex = nullptr;
        if (rc != EFQAT_OK) return rc;
        tiles += t1;
        if (g1 > dx_grid) dx_grid = g1;
      }
    } else {
      // One launch per class of input pixels (a single class for stride 1).  Classes that no
      // filter tap reaches (a 1x1 filter with stride 2 reads one pixel in four) get no launch:
      // their gradient is zero, written by one fill of dX beforehand.
      if (layer->stride > 1 && (layer->R < layer->stride || layer->S < layer->stride)) {
        if (cudaMemsetAsync(dX, 0, static_cast<size_t>(x_elems(layer)) * (act_bf16 ? 2 : 4), st) != cudaSuccess)
          return EFQAT_ERR_CUDA;
      }
      for (int ah = 0; ah < layer->stride; ++ah)
        for (int aw = 0; aw < layer->stride; ++aw) {
          cv_dx.cls_h = ah;
          cv_dx.cls_w = aw;
          g.partials = w.dxpart + 2 * static_cast<int64_t>(tiles);
          g.partials_cap = dx_partials(layer) - tiles;
        g.partials_cap = dx_partials(layer) - tiles;
          int t1 = 0, g1 = 0;
          rc = timed_gemm(ctx, 1, g, st, &t1, &g1);
          if (rc != EFQAT_OK) return rc;
          tiles += t1;
          if (g1 > dx_grid) dx_grid = g1;
        }
    }
  }
  // a6: weight gradient of the unfrozen channels only, as split partial products
  if (k_sel > 0) {
    GemmArgs g = {};
    if (sconv) g.conv = &cv_dw;
    g.A = w.Xc;                       // D[k, i] = sum_m Xc[m,k] * dYsel[m,i]
    g.B = gathered ? w.dYsel : dYb;
    g.Mr = K; g.Nc = gathered ? round_up(k_sel, 16) : N; g.Kc = M;
    g.lda = K; g.ldb = gathered ? w.pitch : N;
    g.a_mn = 1; g.b_mn = 1;
    g.epi = EPI_PART;
    g.out = w.P; g.ldo = K;
    // The weight-gradient GEMM starts beside the grad-input GEMM (defer_wait below).  When the
    // SMs that GEMM leaves idle can hold one CTA per output tile, the contraction is split only
    // as far as those SMs go: every CTA then runs at once and the finalize launch sums fewer
    // partial products.  Otherwise the split sized for the whole GPU stands.
    int splits = w.splits;
    if (!sconv) {
      const int64_t dw_tiles = gemm_part_tiles(g.Mr, g.Nc);
      const int64_t idle = ctx->sm_count - dx_grid;
      if (idle >= dw_tiles && dw_tiles * splits > idle) splits = static_cast<int>(idle / dw_tiles);
      if (splits < 1) splits = 1;
    }
    g.splits = splits;
    dw_splits = splits;
    g.split_stride = k_sel * K;
    g.part_cols = k_sel;
    g.status = ctx->d_status;
    // reads only what the prepare launch wrote, which the grad-input GEMM just before it has
    // already waited for: free to run beside that GEMM on the SMs it leaves idle
    g.defer_wait = 1;
    rc = timed_gemm(ctx, 2, g, st);
    if (rc != EFQAT_OK) return rc;
  }
  // a5 (+ a7): one launch: dW rows (mask, dS_w, optional SGD), dS_x / dZ_x, db
  FinArgs fa = {};
  fa.N = N; fa.K = K; fa.k_sel = k_sel;
  fa.P = w.P; fa.splits = dw_splits; fa.split_stride = k_sel * K;
  fa.W = W; fa.s_w = s_w; fa.s_x = s_x; fa.w_bits = q->w_bits;
  fa.idx = gathered ? idx : nullptr;
  fa.dW_sel = dW_sel; fa.dS_w_sel = dS_w_sel;
  if (opt_or_null) fa.opt = *opt_or_null;
  fa.has_opt = opt_or_null != nullptr;
  fa.dx_partials = w.dxpart; fa.n_partials = tiles; fa.dS_x = dS_x; fa.dZ_x = dZ_x;
  fa.colsum_ws = w.colsum; fa.slabs = prepare_slabs(M, N); fa.db = db_or_null;
  fa.status = ctx->d_status;
  if (chain && chain->defer && fin_is_light(fa)) {
    chain->pending = fa;
    chain->has_pending = true;
  } else {
    launch_finalize(fa, st);
  }
  return last_error();
}

}  // namespace

extern "C" {

int efqat_fq_linear_fwd(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* X,
                        const float* W, const float* s_w, const float* s_x, const float* z_x,
                        const float* bias_or_null, void* Y, void* ws, size_t ws_bytes, efqat_stream_t stream) {
  if (!W) return EFQAT_ERR_NULL;
  return fwd_impl(ctx, layer, q, X, W, s_w, s_x, z_x, bias_or_null, Y, ws, ws_bytes, nullptr, 0, stream);
}

int efqat_fq_linear_bwd(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* dY,
                        const void* X, const float* W, const float* s_w, const float* s_x, const float* z_x,
                        const int32_t* idx, int64_t k_sel, void* dX, float* dW_sel, float* dS_w_sel,
                        float* dS_x, float* dZ_x, float* db_or_null, const efqat_sgd* opt_or_null, void* ws,
                        size_t ws_bytes, efqat_stream_t stream) {
  return bwd_impl(ctx, layer, q, dY, X, W, s_w, s_x, z_x, idx, k_sel, dX, dW_sel, dS_w_sel, dS_x, dZ_x, db_or_null,
                  opt_or_null, ws, ws_bytes, nullptr, 0, stream);
}

int efqat_weight_cache_bytes(const efqat_layer_desc* layer, const efqat_qspec* q, size_t* out) {
  if (!out) return EFQAT_ERR_NULL;
  const int rc = check_layer(layer, q);
  if (rc != EFQAT_OK) return rc;
  *out = carve_cache(nullptr, layer).bytes;
  return EFQAT_OK;
}

int efqat_weight_cache_update(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const float* W,
                              const float* s_w, const int32_t* idx, int64_t k_sel, void* cache, size_t cache_bytes,
                              efqat_stream_t stream) {
  if (!ctx || !W || !s_w || !cache) return EFQAT_ERR_NULL;
  int rc = check_layer(layer, q);
  if (rc != EFQAT_OK) return rc;
  if (k_sel < 0 || k_sel > layer->N) return EFQAT_ERR_K_RANGE;
  if (k_sel > 0 && k_sel < layer->N && !idx) return EFQAT_ERR_NULL;
  if (!aligned16(W)) return EFQAT_ERR_ALIGN;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  const WCache wc = carve_cache(cache, layer);
  if (cache_bytes < wc.bytes) return EFQAT_ERR_WORKSPACE;
  Entered in(ctx);
  CacheArgs a = {};
  a.N = layer->N; a.K = layer->K; a.rows = k_sel;
  a.W = W; a.s_w = s_w; a.w_bits = q->w_bits;
  a.idx = (k_sel < layer->N) ? idx : nullptr;
  a.codes8 = wc.codes8; a.wsum = wc.wsum; a.codes16 = wc.codes16; a.what = wc.what;
  a.status = ctx->d_status;
  launch_weight_cache(a, stream);
  return last_error();
}

int efqat_fq_linear_fwd_cached(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* X,
                               const float* s_w, const float* s_x, const float* z_x, const float* bias_or_null,
                               void* Y, const void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               efqat_stream_t stream) {
  if (!cache) return EFQAT_ERR_NULL;
  return fwd_impl(ctx, layer, q, X, nullptr, s_w, s_x, z_x, bias_or_null, Y, ws, ws_bytes, cache, cache_bytes, stream);
}

int efqat_fq_linear_bwd_cached(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* dY,
                               const void* X, const float* W, const float* s_w, const float* s_x, const float* z_x,
                               const int32_t* idx, int64_t k_sel, void* dX, float* dW_sel, float* dS_w_sel,
                               float* dS_x, float* dZ_x, float* db_or_null, const efqat_sgd* opt_or_null,
                               const void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               efqat_stream_t stream) {
  if (!cache) return EFQAT_ERR_NULL;
  return bwd_impl(ctx, layer, q, dY, X, W, s_w, s_x, z_x, idx, k_sel, dX, dW_sel, dS_w_sel, dS_x, dZ_x, db_or_null,
                  opt_or_null, ws, ws_bytes, cache, cache_bytes, stream);
}

int efqat_network_fwd(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream) {
  if (!ctx || !layers) return EFQAT_ERR_NULL;
  if (L < 1) return EFQAT_ERR_SHAPE;
  for (int l = 0; l < L; ++l) {
    const efqat_net_layer& n = layers[l];
    const int rc = fwd_impl(ctx, &n.layer, &n.q, n.X, n.W, n.s_w, n.s_x, n.z_x, n.bias_or_null, n.Y, n.ws, n.ws_bytes,
                            n.cache_or_null, n.cache_bytes, stream);
    if (rc != EFQAT_OK) return rc;
  }
  return EFQAT_OK;
}

int efqat_network_bwd(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream) {
  if (!ctx || !layers) return EFQAT_ERR_NULL;
  if (L < 1) return EFQAT_ERR_SHAPE;
  // A layer's finalize work rides in the prepare launch of the layer processed next whenever the two
  // layers' workspaces are disjoint (the prepare jobs write theirs while the finalize blocks read the
  // other); layers that share a workspace keep one finalize launch each.
  FinChain ch = {};
  for (int l = L - 1; l >= 0; --l) {
    const efqat_net_layer& n = layers[l];
    ch.defer = false;
    if (l > 0) {
      const efqat_net_layer& m = layers[l - 1];
      const char* a0 = static_cast<const char*>(n.ws);
      const char* b0 = static_cast<const char*>(m.ws);
      ch.defer = n.ws && m.ws && (a0 + n.ws_bytes <= b0 || b0 + m.ws_bytes <= a0) && n.W != m.W;
    }
    const int rc = bwd_impl(ctx, &n.layer, &n.q, n.dY, n.X, n.W, n.s_w, n.s_x, n.z_x, n.idx, n.k_sel, n.dX, n.dW_sel,
                            n.dS_w_sel, n.dS_x, n.dZ_x, n.db_or_null, n.opt_or_null, n.ws, n.ws_bytes,
                            n.cache_or_null, n.cache_bytes, stream, &ch);
    if (rc != EFQAT_OK || l == 0) {
      if (ch.has_pending) {          // a layer's call failed before its prepare launch: the work still pending goes out alone
        if (guard_device(ctx) == EFQAT_OK) launch_finalize(ch.pending, stream);
        ch.has_pending = false;
      }
      if (rc != EFQAT_OK) return rc;
    }
  }
  return last_error();
}

int efqat_network_cache_update(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream) {
  if (!ctx || !layers) return EFQAT_ERR_NULL;
  if (L < 1) return EFQAT_ERR_SHAPE;
  for (int l = 0; l < L; ++l) {
    const efqat_net_layer& n = layers[l];
    if (!n.cache_or_null || n.k_sel == 0) continue;
    const int rc = efqat_weight_cache_update(ctx, &n.layer, &n.q, n.W, n.s_w, n.idx, n.k_sel, n.cache_or_null,
                                             n.cache_bytes, stream);
    if (rc != EFQAT_OK) return rc;
  }
  return EFQAT_OK;
}

int efqat_gemm_bf16(efqat_ctx* ctx, const void* A, const void* B, int64_t M, int64_t N, int64_t K, int a_mn,
                    int b_mn, int splits, float* out, efqat_stream_t stream) {
  if (!ctx || !A || !B || !out) return EFQAT_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || splits < 1) return EFQAT_ERR_SHAPE;
  if ((M & 7) || (N & 7) || (K & 7)) return EFQAT_ERR_ALIGN;
  if (!aligned16(A) || !aligned16(B) || !aligned16(out)) return EFQAT_ERR_ALIGN;
  int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  GemmArgs g = {};
  g.A = static_cast<const bf16*>(A); g.B = static_cast<const bf16*>(B);
  g.Mr = M; g.Nc = N; g.Kc = K;
  g.lda = a_mn ? M : K; g.ldb = b_mn ? N : K;
  g.a_mn = a_mn ? 1 : 0; g.b_mn = b_mn ? 1 : 0;
  g.epi = EPI_PART;
  g.out = out; g.ldo = M;
  g.splits = splits;
  g.split_stride = M * N;
  g.part_cols = N;
  g.status = ctx->d_status;
  rc = run_gemm(g, ctx->sm_count, stream);
  if (rc != EFQAT_OK) return rc;
  return last_error();
}

int efqat_qparam_adam(efqat_ctx* ctx, const efqat_adam* opt, const efqat_qparam_state* state, int64_t N,
                      const int32_t* idx, int64_t k_sel, const float* dS_w_sel, const float* dS_x,
                      const float* dZ_x, efqat_stream_t stream) {
  if (!ctx || !opt || !state || !dS_x || !state->s_x || !state->state_x) return EFQAT_ERR_NULL;
  if (N < 1) return EFQAT_ERR_SHAPE;
  if (k_sel < 0 || k_sel > N) return EFQAT_ERR_K_RANGE;
  if (k_sel > 0 && (!dS_w_sel || !state->s_w || !state->m_sw || !state->v_sw)) return EFQAT_ERR_NULL;
  if (k_sel > 0 && k_sel < N && !idx) return EFQAT_ERR_NULL;
  if (opt->log2_scale && k_sel > 0 && !state->theta_sw) return EFQAT_ERR_NULL;
  if (dZ_x && !state->z_x) return EFQAT_ERR_NULL;
  if (opt->step < 1 || !(opt->beta1 >= 0.f && opt->beta1 < 1.f) || !(opt->beta2 >= 0.f && opt->beta2 < 1.f) ||
      !(opt->eps > 0.f))
    return EFQAT_ERR_SHAPE;
  const int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_qparam_adam(*opt, *state, N, (k_sel < N) ? idx : nullptr, k_sel, dS_w_sel, dS_x, dZ_x, ctx->d_status, stream);
  return last_error();
}

int efqat_network_qparam_adam(efqat_ctx* ctx, const efqat_adam* opt, int L, const efqat_net_layer* layers,
                              const efqat_qparam_state* states, efqat_stream_t stream) {
  if (!ctx || !opt || !layers || !states) return EFQAT_ERR_NULL;
  if (L < 1) return EFQAT_ERR_SHAPE;
  for (int l = 0; l < L; ++l) {
    const efqat_net_layer& n = layers[l];
    const int rc = efqat_qparam_adam(ctx, opt, &states[l], n.layer.N, n.idx, n.k_sel, n.dS_w_sel, n.dS_x,
                                     n.q.x_symmetric ? nullptr : n.dZ_x, stream);
    if (rc != EFQAT_OK) return rc;
  }
  return EFQAT_OK;
}

int efqat_log2_scale_init(efqat_ctx* ctx, const float* s, float* theta, int64_t n, efqat_stream_t stream) {
  if (!ctx || !s || !theta) return EFQAT_ERR_NULL;
  if (n < 1) return EFQAT_ERR_SHAPE;
  const int rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_log2_init(s, theta, n, ctx->d_status, stream);
  return last_error();
}

int efqat_fake_quant_act(efqat_ctx* ctx, const efqat_qspec* q, int dtype, const void* x, int64_t count,
                         const float* s_x, const float* z_x, int32_t* codes_or_null, uint8_t* clip_or_null,
                         efqat_stream_t stream) {
  if (!ctx || !x || !s_x) return EFQAT_ERR_NULL;
  int rc = check_bits(q);
  if (rc != EFQAT_OK) return rc;
  if (!q->x_symmetric && !z_x) return EFQAT_ERR_NULL;
  if (dtype != EFQAT_F32 && dtype != EFQAT_BF16) return EFQAT_ERR_DTYPE;
  if (count < 0) return EFQAT_ERR_SHAPE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  ActQ* scratch = reinterpret_cast<ActQ*>(reinterpret_cast<char*>(ctx->d_status) + 128);
  launch_prep_act(s_x, z_x, q->x_bits, q->x_symmetric, scratch, ctx->d_status, stream);
  launch_quant_act_export(x, dtype, count, scratch, codes_or_null, clip_or_null, stream);
  return last_error();
}

int efqat_fake_quant_weight(efqat_ctx* ctx, const efqat_qspec* q, const float* W, int64_t N, int64_t K,
                            const float* s_w, int32_t* codes_or_null, uint8_t* clip_or_null,
                            efqat_stream_t stream) {
  if (!ctx || !W || !s_w) return EFQAT_ERR_NULL;
  int rc = check_bits(q);
  if (rc != EFQAT_OK) return rc;
  if (N < 0 || K < 1) return EFQAT_ERR_SHAPE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_quant_weight_export(W, N, K, s_w, q->w_bits, codes_or_null, clip_or_null, ctx->d_status, stream);
  return last_error();
}

int efqat_init_act_qparams(efqat_ctx* ctx, const efqat_qspec* q, int dtype, const void* x, int64_t count,
                           float* s_x, float* z_x, void* ws, size_t ws_bytes, efqat_stream_t stream) {
  if (!ctx || !x || !s_x || !z_x) return EFQAT_ERR_NULL;
  int rc = check_bits(q);
  if (rc != EFQAT_OK) return rc;
  if (dtype != EFQAT_F32 && dtype != EFQAT_BF16) return EFQAT_ERR_DTYPE;
  if (count < 1) return EFQAT_ERR_SHAPE;
  if (!ws || ws_bytes < 8192) return EFQAT_ERR_WORKSPACE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_minmax_act(x, dtype, count, q->x_bits, q->x_symmetric, s_x, z_x, static_cast<float*>(ws), stream);
  return last_error();
}

int efqat_init_weight_scales(efqat_ctx* ctx, const efqat_qspec* q, const float* W, int64_t N, int64_t K,
                             float* s_w, efqat_stream_t stream) {
  if (!ctx || !W || !s_w) return EFQAT_ERR_NULL;
  int rc = check_bits(q);
  if (rc != EFQAT_OK) return rc;
  if (N < 1 || K < 1) return EFQAT_ERR_SHAPE;
  rc = guard_device(ctx);
  if (rc != EFQAT_OK) return rc;
  Entered in(ctx);
  launch_absmax_rows(W, N, K, q->w_bits, s_w, stream);
  return last_error();
}

}  // extern "C"
