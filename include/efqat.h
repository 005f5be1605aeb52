/*
 * efqat.h -- C ABI of the B200 (sm_100a) library for the EfQAT training step of a
 * fake-quantized linear / convolution layer (EfQAT, arxiv 2411.11038).
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless a parameter is
 *     documented as "host".  The library never frees or keeps caller memory.
 *   - Calls enqueue work on `stream` and return without synchronising.  Scratch memory
 *     comes from the caller-provided workspace `ws` (size it with the *_workspace_bytes
 *     queries); nothing is allocated on the hot path.
 *   - Return value: 0 (EFQAT_OK) or a negative efqat_status found on the host before any
 *     launch.  Conditions only the device can see (a non-positive or non-finite scale, an
 *     index out of range, a bounded wait that ran out) are recorded in a context-owned
 *     status word read with efqat_device_status() after the caller synchronised.
 *   - Layouts: row-major.  Linear: X[M,K], W[N,K], Y/dY[M,N] (PyTorch Linear convention,
 *     paper Section 3.1 footnote).  Convolution: X NHWC [B,H,W,Cin], W [N,R,S,Cin],
 *     Y/dY [B,Ho,Wo,N]; its GEMM view is M = B*Ho*Wo, K = R*S*Cin.
 *   - Alignment: every base pointer 16-byte aligned; N % 8 == 0 and K % 8 == 0 (Cin % 8 == 0
 *     for convolutions: an input with fewer channels, such as a 3-channel image, is stored
 *     with zero channels up to 8, and so is its filter).  Violations return EFQAT_ERR_ALIGN;
 *     there is no slow path.
 *   - Activations (X, dY, Y, dX) are fp32 or bf16 (efqat_dtype); weights, scales, zero
 *     point, bias and all gradients of parameters are fp32.
 */
#ifndef EFQAT_H_
#define EFQAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct efqat_ctx efqat_ctx;          /* opaque: device, SM count, status word */
typedef struct CUstream_st* efqat_stream_t;  /* same type as cudaStream_t / CUstream */

typedef enum {
  EFQAT_OK = 0,
  EFQAT_ERR_NULL = -1,       /* a required pointer is NULL */
  EFQAT_ERR_SHAPE = -2,      /* a dimension is < 1 or inconsistent */
  EFQAT_ERR_ALIGN = -3,      /* pointer or pitch alignment contract violated */
  EFQAT_ERR_DTYPE = -4,      /* unknown efqat_dtype */
  EFQAT_ERR_BITS = -5,       /* bit-width outside [2,8] */
  EFQAT_ERR_MODE = -6,       /* unknown efqat_mode */
  EFQAT_ERR_WORKSPACE = -7,  /* workspace too small or NULL */
  EFQAT_ERR_K_RANGE = -8,    /* k_sel / budget outside its range */
  EFQAT_ERR_UNIMPL = -9,     /* combination not built (e.g. conv stride > 2, filter beyond 7 x 7) */
  EFQAT_ERR_CUDA = -10,      /* a CUDA runtime / driver call failed */
  EFQAT_ERR_TOO_LARGE = -11, /* a size exceeds a fixed built-in maximum (efqat_colsum_noalloc) */
  /* device-side conditions, reported by efqat_device_status (positive) */
  EFQAT_DEV_BAD_SCALE = 1,   /* a scale was <= 0 or not finite */
  EFQAT_DEV_BAD_INDEX = 2,   /* idx entry outside [0,N) or not strictly ascending */
  EFQAT_DEV_WAIT_TIMEOUT = 3 /* a bounded in-kernel wait expired */
} efqat_status;

/* Table 2 of the paper: freezing granularity x selection scope. */
typedef enum { EFQAT_CWPL = 0, EFQAT_CWPN = 1, EFQAT_LWPN = 2 } efqat_mode;
typedef enum { EFQAT_F32 = 0, EFQAT_BF16 = 1 } efqat_dtype;

/* Bit-widths b of Eq. 1 / Eq. 3.  Weights are always symmetric per output channel
 * (Eq. 3-4); activations are per tensor, asymmetric (Eq. 1-2) unless x_symmetric != 0,
 * in which case Z = 0 and the code range is [-(2^(b-1)-1), 2^(b-1)-1]. */
typedef struct {
  int w_bits;
  int x_bits;
  int x_symmetric;
} efqat_qspec;

/* One quantized layer.  Linear: is_conv = 0 and only M, N, K, act_dtype are read.
 * Convolution: is_conv = 1, stride 1 or 2 (the same along H and W), filters up to 7 x 7
 * (R*S <= 49), pad < R and pad < S, Ho = (H + 2*pad - R) / stride + 1 (Wo alike); M and K must
 * equal B*Ho*Wo and R*S*Cin.  This covers the paper's networks: 1x1 and 3x3 convolutions, the
 * stride-2 3x3 and 1x1 shortcut convolutions and the 7x7 stride-2 input layer (Section 4). */
typedef struct {
  int64_t M, N, K;
  int is_conv;
  int B, H, W, Cin, R, S, stride, pad;
  int act_dtype; /* efqat_dtype of X, dY, Y, dX */
} efqat_layer_desc;

/* Optional fused optimizer for the unfrozen rows (Algorithm 1, optimizer step; SGD with
 * momentum as in the paper's Section 4): v <- momentum*v + (g + weight_decay*w);
 * w <- w - lr*v on rows idx[] of W_inout / mom_inout (both fp32 [N,K]); other rows are
 * never touched. */
typedef struct {
  float lr, momentum, weight_decay;
  float* W_inout;
  float* mom_inout;
} efqat_sgd;

/* ---- context ------------------------------------------------------------------- */
/* Creates a context bound to CUDA device `device` (allocates a few hundred bytes of
 * device memory for the status word; the only allocation the library ever makes). */
int efqat_create(efqat_ctx** out, int device);
int efqat_destroy(efqat_ctx* ctx);
/* Static, human-readable name of a status code (host or device side). */
const char* efqat_status_string(int status);
/* Reads and clears the device status word.  Synchronises the device; call it after the
 * stream work of interest was enqueued.  *code = 0 or an EFQAT_DEV_* value. */
int efqat_device_status(efqat_ctx* ctx, int* code);

/* ---- host-only helpers ---------------------------------------------------------- */
/* floor(ratio * n): number of unfrozen channels for ratio r (Eq. 7). */
int64_t efqat_ratio_to_k(double ratio, int64_t n);
/* Checks a layer description + quantizer spec exactly as the compute calls do. */
int efqat_validate_layer(const efqat_layer_desc* layer, const efqat_qspec* q);
/* Workspace bytes for efqat_fq_linear_fwd / _bwd on `layer` with at most k_sel_max
 * selected channels (pass N to cover full-QAT).  The size depends on the SM count of the
 * GPU: the query reads it from the current CUDA device, which must be the device the
 * compute calls will run on (they require their context's device to be current too). */
int efqat_workspace_bytes(const efqat_layer_desc* layer, const efqat_qspec* q, int64_t k_sel_max, size_t* out);
/* Workspace bytes for efqat_select_channels over L layers with total_channels rows. */
int efqat_select_workspace_bytes(int L, int64_t total_channels, size_t* out);

/* ---- a1: importance + Top-K selection (Eq. 6, Table 2, Algorithm 1 "extract the unfrozen
 * channels") ---------------------------------------------------------------------- */
/* layers[l].N / .K give the shape of weights[l] (fp32 [N_l, K_l], device); `layers`,
 * `weights` (array of device pointers) and `k` are HOST arrays of length L.
 *   CWPL: k[l] channels are kept in layer l (0 <= k[l] <= N_l).
 *   CWPN: k[0] = channel budget over the whole network; one ranking of all channels by
 *         importance, ties to the smaller (layer, channel).
 *   LWPN: k[0] = number of layers kept; layers ranked by mean |w| over the whole layer;
 *         a kept layer has every channel selected.
 * Ranking: larger mean |w| first, ties to the smaller index.
 * Outputs (device): idx int32, concatenated per layer, ascending inside a layer (capacity:
 * sum of k for CWPL, k[0] for CWPN, total_channels for LWPN); offsets int32 [L+1] with
 * layer l owning idx[offsets[l] .. offsets[l+1]); importance_or_null fp32 keys
 * (concatenated channels for CWPL/CWPN, one per layer for LWPN). */
int efqat_select_channels(efqat_ctx* ctx, int mode, int L, const efqat_layer_desc* layers,
                          const float* const* weights, const int64_t* k, int32_t* idx, int32_t* offsets,
                          float* importance_or_null, void* ws, size_t ws_bytes, efqat_stream_t stream);

/* ---- a2 + a3: fake-quantize X and W, forward GEMM (Eq. 1, Eq. 3, Section 3.1) -------- */
/* Y[m,n] = s_x * s_w[n] * sum_k (q_x[m,k] - Z) * q_w[n,k] + bias[n].
 * s_w [N], s_x [1], z_x [1] (ignored when x_symmetric), bias [N] or NULL; Y in act_dtype.
 * Plain layers with 512 <= K <= 32768, K % 16 == 0 and N % 32 == 0 contract the 8-bit codes
 * on the integer tensor cores (int32 accumulation: the integer sum is exact); all others
 * contract the same integers held in bf16, with fp32 accumulation.  Plain layers with K = 64
 * (and, for bf16 activations, K = 128) and N % 64 == 0 run in a single launch that reads X
 * and writes Y once. */
int efqat_fq_linear_fwd(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* X,
                        const float* W, const float* s_w, const float* s_x, const float* z_x,
                        const float* bias_or_null, void* Y, void* ws, size_t ws_bytes, efqat_stream_t stream);

/* ---- a4 + a5 + a6 (+ a7): backward (Eq. 5, Algorithm 1, straight-through estimator) --- */
/* Always: dX = (dY W^) * [x not clipped]  (act_dtype, shape of X), dS_x [1], dZ_x [1],
 * db_or_null [N] = column sums of dY.
 * Unfrozen channels only: idx [k_sel] ascending device int32 (may be NULL when k_sel == 0
 * or k_sel == N); dW_sel fp32 [k_sel, K] with row i <-> channel idx[i];
 * dS_w_sel fp32 [k_sel].  k_sel == N is the ordinary QAT backward; k_sel == 0 does no
 * weight-gradient work at all.  dW_sel carries the weight quantizer's clip mask.
 * opt_or_null != NULL applies the fused SGD-momentum update to rows idx of opt->W_inout.
 * Plain bf16 layers with K = 64 and N = 128 or 256 take a one-pass form that reads dY and X
 * once whatever k_sel is. */
int efqat_fq_linear_bwd(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* dY,
                        const void* X, const float* W, const float* s_w, const float* s_x, const float* z_x,
                        const int32_t* idx, int64_t k_sel, void* dX, float* dW_sel, float* dS_w_sel,
                        float* dS_x, float* dZ_x, float* db_or_null, const efqat_sgd* opt_or_null, void* ws,
                        size_t ws_bytes, efqat_stream_t stream);

/* ---- weight-operand cache and whole-network calls (Section 3.2 "Freezing Frequency";
 * Algorithm 1 runs the layer step over every layer of the network) --------------------- */
/* Between two selections the frozen channels keep their weights and scales, hence their
 * integer codes.  A caller-owned cache per layer holds the quantized weight operands of both
 * passes (forward: the codes; backward: the dequantised weights of the grad-input GEMM), so
 * that a forward / backward no longer reads W or re-quantizes it; after an optimizer step
 * only the rows that step touched are rebuilt.  A cached operand is bit-identical to the one
 * the uncached calls build, as long as every row whose weights or scale changed since its
 * last rebuild is passed to efqat_weight_cache_update before the next cached call: keeping it
 * current is the caller's contract, nothing in the block records validity. */
/* Bytes of the cache block of `layer` (device memory, any alignment). */
int efqat_weight_cache_bytes(const efqat_layer_desc* layer, const efqat_qspec* q, size_t* out);
/* Rebuilds rows idx[0..k_sel) of the cache from W fp32 [N,K] and s_w [N] (k_sel == N: every
 * row, idx may be NULL; k_sel == 0: nothing).  idx: device int32, ascending, as returned by
 * efqat_select_channels.  Call it once with k_sel = N before the first cached call. */
int efqat_weight_cache_update(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const float* W,
                              const float* s_w, const int32_t* idx, int64_t k_sel, void* cache, size_t cache_bytes,
                              efqat_stream_t stream);
/* efqat_fq_linear_fwd with the weight operand taken from the cache: W is not read. */
int efqat_fq_linear_fwd_cached(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* X,
                               const float* s_w, const float* s_x, const float* z_x, const float* bias_or_null,
                               void* Y, const void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               efqat_stream_t stream);
/* efqat_fq_linear_bwd with the grad-input operand taken from the cache; W is read only on the
 * unfrozen rows (clip mask, dS_w, fused SGD). */
int efqat_fq_linear_bwd_cached(efqat_ctx* ctx, const efqat_layer_desc* layer, const efqat_qspec* q, const void* dY,
                               const void* X, const float* W, const float* s_w, const float* s_x, const float* z_x,
                               const int32_t* idx, int64_t k_sel, void* dX, float* dW_sel, float* dS_w_sel,
                               float* dS_x, float* dZ_x, float* db_or_null, const efqat_sgd* opt_or_null,
                               const void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               efqat_stream_t stream);

/* One layer of a network: the arguments of the layer calls above, gathered (HOST struct, device
 * pointers inside, meanings as documented there).  cache_or_null == NULL selects the uncached
 * calls.  Layers may share one workspace `ws` (sized for the largest): the calls are ordered
 * on the stream. */
typedef struct {
  efqat_layer_desc layer;
  efqat_qspec q;
  const void* X; const float* W; const float* s_w; const float* s_x; const float* z_x;
  const float* bias_or_null; void* Y;                                   /* forward */
  const void* dY; const int32_t* idx; int64_t k_sel;                    /* backward */
  void* dX; float* dW_sel; float* dS_w_sel; float* dS_x; float* dZ_x; float* db_or_null;
  const efqat_sgd* opt_or_null;
  void* cache_or_null; size_t cache_bytes;
  void* ws; size_t ws_bytes;
} efqat_net_layer;
/* Forward of layers[0..L) in order / backward of layers[L-1..0] in reverse order, enqueued on
 * one stream with no host synchronisation in between (each launch overlaps its set-up with
 * the tail of the one before it).  Stops at, and returns, the first host-side error.
 * Layers may share one workspace; when neighbouring layers have disjoint workspaces (two buffers
 * taken in turn are enough) the backward saves a launch per layer: a layer's last launch (the
 * reduction of its partial sums, masks, optional SGD) then shares a launch with the first one of
 * the layer processed next.  Results are the same bits either way. */
int efqat_network_fwd(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream);
int efqat_network_bwd(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream);
/* efqat_weight_cache_update on rows idx of every layer that has a cache and k_sel > 0 (after
 * the optimizer steps of a training step). */
int efqat_network_cache_update(efqat_ctx* ctx, int L, const efqat_net_layer* layers, efqat_stream_t stream);

/* ---- optimizer step of the quantization parameters (Section 4 "Setup": Adam for the
 * quantization parameters; Algorithm 1: "update the unfrozen weight channels and their
 * scales", "update the scales and zero points of the activations"; Appendix A.2: optional
 * log2 parameterisation of the scales) --------------------------------------------------- */
/* Adam:  m <- beta1 m + (1-beta1) g;  v <- beta2 v + (1-beta2) g^2;
 *        p <- p - lr (m / (1-beta1^step)) / (sqrt(v / (1-beta2^step)) + eps),  step >= 1.
 * log2_scale != 0: for the scales the optimised variable is theta = log2(s), with gradient
 * g * s * ln 2, and s <- 2^theta afterwards; the zero point is always trained raw. */
typedef struct {
  float lr, beta1, beta2, eps;
  int64_t step;
  int log2_scale;
} efqat_adam;
/* Parameters and optimizer state of one layer (device, fp32, caller-owned).  s_w, m_sw, v_sw,
 * theta_sw: [N] (theta_sw only used, and required, in log2 mode: initialise it with
 * efqat_log2_scale_init).  s_x, z_x: [1].  state_x: [8] = first and second moment of s_x,
 * first and second moment of z_x, theta of s_x, three unused; zero it before the first step
 * (and set element 4 with efqat_log2_scale_init in log2 mode). */
typedef struct {
  float* s_w; float* m_sw; float* v_sw; float* theta_sw;
  float* s_x; float* z_x; float* state_x;
} efqat_qparam_state;
/* One launch: the weight scales of the channels idx[0..k_sel) (idx may be NULL when
 * k_sel == N; scales and moments of the other channels are not touched) from the compact
 * gradient dS_w_sel [k_sel], the activation scale from dS_x [1], and the activation zero
 * point from dZ_x [1] (dZ_x NULL, e.g. for the symmetric quantizer: zero point left alone).
 * The gradients are the outputs of efqat_fq_linear_bwd.  A raw scale that the step drives
 * to zero or below is reported as EFQAT_DEV_BAD_SCALE by the next forward / backward. */
int efqat_qparam_adam(efqat_ctx* ctx, const efqat_adam* opt, const efqat_qparam_state* state, int64_t N,
                      const int32_t* idx, int64_t k_sel, const float* dS_w_sel, const float* dS_x,
                      const float* dZ_x, efqat_stream_t stream);
/* efqat_qparam_adam over the layers of a network in one call (HOST arrays of length L: the
 * per-layer states; layers[l] supplies N, idx, k_sel, dS_w_sel, dS_x, dZ_x; a layer with the
 * symmetric activation quantizer leaves its zero point alone). */
int efqat_network_qparam_adam(efqat_ctx* ctx, const efqat_adam* opt, int L, const efqat_net_layer* layers,
                              const efqat_qparam_state* states, efqat_stream_t stream);
/* theta[i] = log2(s[i]) for i < n (Appendix A.2). */
int efqat_log2_scale_init(efqat_ctx* ctx, const float* s, float* theta, int64_t n, efqat_stream_t stream);

/* ---- helpers: quantizer export and MinMax initialisation ---------------------------- */
/* Eq. 1: codes int32 [count] (asymmetric: 0..2^b-1; symmetric: signed), clip uint8 [count]
 * (0 in range, 1 clipped low, 2 clipped high), either may be NULL.  x in `dtype`. */
int efqat_fake_quant_act(efqat_ctx* ctx, const efqat_qspec* q, int dtype, const void* x, int64_t count,
                         const float* s_x, const float* z_x, int32_t* codes_or_null, uint8_t* clip_or_null,
                         efqat_stream_t stream);
/* Eq. 3: W fp32 [N,K] with per-row scales s_w [N]; codes int32 [N,K], clip uint8 [N,K]. */
int efqat_fake_quant_weight(efqat_ctx* ctx, const efqat_qspec* q, const float* W, int64_t N, int64_t K,
                            const float* s_w, int32_t* codes_or_null, uint8_t* clip_or_null,
                            efqat_stream_t stream);
/* Eq. 2 (activations, per tensor; symmetric variant when q->x_symmetric) -> s_x[1], z_x[1].
 * ws: at least 8192 bytes. */
int efqat_init_act_qparams(efqat_ctx* ctx, const efqat_qspec* q, int dtype, const void* x, int64_t count,
                           float* s_x, float* z_x, void* ws, size_t ws_bytes, efqat_stream_t stream);
/* Eq. 4 (weights, per output channel) -> s_w[N]. */
int efqat_init_weight_scales(efqat_ctx* ctx, const efqat_qspec* q, const float* W, int64_t N, int64_t K,
                             float* s_w, efqat_stream_t stream);

/* ---- allocation-free bias gradient ------------------------------------------------- */
/* The paper has no counterpart to this call; it exists for integration reasons only.
 * db[n] = sum_m dY[m,n] (fp32), the same column sums efqat_fq_linear_bwd writes to
 * db_or_null, for callers that cannot allocate device memory at all and therefore can
 * neither create a context nor provide a workspace: an enqueue hook of a runtime that hands
 * out a fixed arena and forbids further allocation, a latency-critical loop that must not
 * enter the allocator, a process whose device memory pool belongs to another component.
 * The partial sums live in a 4 MiB device array built into the library (held on every
 * GPU that loads it, for the life of the process).  Needs no efqat_ctx.  The call itself
 * calls no allocating routine and frees nothing.
 *   dY: device, [M,N] row-major in `dtype` (EFQAT_F32 / EFQAT_BF16), 16-byte aligned;
 *   db: device, fp32 [N];  N % 8 == 0 and N <= 16384, else EFQAT_ERR_ALIGN /
 *   EFQAT_ERR_TOO_LARGE; the CUDA device owning dY must be current.
 * The first call on each device is a warm-up: it looks up the array's device address, and
 * under CUDA's lazy module loading the runtime may load this library's device code (the
 * array included) at that moment, which takes device memory.  Make that first call before
 * entering the region in which nothing may be allocated, and before starting any stream
 * capture.  All calls share the one array and it keeps what the previous call left there
 * (each call overwrites every element it reads, so nothing needs clearing), hence two calls
 * whose kernels may overlap on the GPU -- different streams without ordering -- race with
 * each other: serialise them. */
int efqat_colsum_noalloc(int dtype, const void* dY, int64_t M, int64_t N, float* db, efqat_stream_t stream);

/* ---- helper: the tensor-core contraction shared by a3, a4 and a6 (Eq. 5 shapes) -------- */
/* out[n*M + m] = sum_k A(m,k) * B(n,k) in fp32, bf16 operands (device), i.e. the product is
 * written transposed, [N,M] row-major, one slab per split: out has splits*N*M floats and
 * the caller adds the slabs.  a_mn = 0: A stored [M,K] row-major; a_mn = 1: A stored [K,M].
 * b_mn = 0: B stored [N,K]; b_mn = 1: B stored [K,N].  M, N, K multiples of 8;
 * 1 <= splits <= ceil(K/64).  Exposed so the four operand layouts can be tested alone. */
int efqat_gemm_bf16(efqat_ctx* ctx, const void* A, const void* B, int64_t M, int64_t N, int64_t K, int a_mn,
                    int b_mn, int splits, float* out, efqat_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* EFQAT_H_ */
