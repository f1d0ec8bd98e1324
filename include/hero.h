/*
 * hero.h - C ABI of the B200 (sm_100a) W8A8 transformer-layer forward of ZeroQuant-HERO.
 *
 * Every pointer named "device" is a CUDA device pointer on the GPU that was current when the
 * handle was created; everything else is host memory or a plain value.  The caller owns every
 * buffer and the stream.  No entry point on the hot path allocates or frees device memory, and
 * every call is asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default stream).
 * Nothing crosses this boundary but plain C types: no exceptions, no abort, no trap.
 *
 * Conventions (paper Sec. 2.1):
 *   - INT8 is symmetric, range [-127, 127]; Round() is round-half-to-even.
 *   - A linear layer is Y = X W with X [n, d] and W [d, m].  Weights are passed "column-major" as
 *     the paper says: an array [m][d] (one output column after another, the reduction dimension d
 *     contiguous), with one scale per output column, S_w [m] (Eq. 2).
 *   - Activation scales follow Eq. 3-5: TWQ S_x [n] (one per token row, computed on the fly by
 *     LN^quant and written by the library), FWQ S_x [d] (calibrated, read by the library),
 *     SQ a single value (device pointer to one float).
 *   - All scale / bias / gamma / beta vectors are device float32.
 *   - Matrices are row-major with a leading dimension `ld` in elements; data pointers must be
 *     16-byte aligned and ld * sizeof(element) a multiple of 16.
 *
 * Errors: every call returns a hero_status.  HERO_ERR_INVALID_ARG / _UNSUPPORTED / _ALIGNMENT are
 * detected on the host before anything is launched.  HERO_ERR_CUDA reports a failed runtime call
 * (text via hero_last_error()).  A device-side wait that exceeded its bound (a pipeline bug, never
 * expected) sets a device error word; hero_check() synchronizes the stream and returns
 * HERO_ERR_DEVICE_TIMEOUT if it is set.  The same word reports an embedding id outside its table (the gather of
 * hero_layernorm_quant clamps such an id, so nothing is read out of bounds): hero_check() then returns
 * HERO_ERR_INVALID_ARG.
 */
#ifndef HERO_H_
#define HERO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HERO_OK = 0,
  HERO_ERR_INVALID_ARG = 1,
  HERO_ERR_UNSUPPORTED = 2,
  HERO_ERR_ALIGNMENT = 3,
  HERO_ERR_WORKSPACE = 4,
  HERO_ERR_CUDA = 5,
  HERO_ERR_DEVICE_TIMEOUT = 6
} hero_status;

/* HERO_F8: e4m3 (1 sign, 4 exponent, 3 mantissa bits, largest finite value 448, no infinities): the payload of the FP8
 * variant of the method (the paper: "the approach carries over to FP8").  An F8 tensor carries scales exactly like an
 * I8 tensor (TWQ / FWQ / SQ); a scale computed on the fly is absmax / 448 and the quantizer is the saturating
 * round-to-nearest-even conversion.  Accepted by hero_layernorm_quant (inputs and output) and hero_w8a8_linear. */
typedef enum { HERO_I8 = 0, HERO_U8 = 1, HERO_I32 = 2, HERO_F16 = 3, HERO_BF16 = 4, HERO_F32 = 5, HERO_F8 = 6 } hero_dtype;

/* Granularity of the scale attached to an INT8 tensor (Eq. 3-5). */
typedef enum { HERO_GRAN_NONE = 0, HERO_GRAN_TWQ = 1, HERO_GRAN_FWQ = 2, HERO_GRAN_SQ = 3 } hero_gran;

typedef enum { HERO_ACT_NONE = 0, HERO_ACT_GELU_ERF = 1, HERO_ACT_GELU_TANH = 2 } hero_act;
typedef enum { HERO_MASK_NONE = 0, HERO_MASK_CAUSAL = 1 } hero_mask;
typedef enum { HERO_POST_LN = 0, HERO_PRE_LN = 1 } hero_arch;
/* Table 1: a module runs INT8 or stays in FP16/BF16 (the layer's fp_dtype). */
typedef enum { HERO_MODE_INT8 = 0, HERO_MODE_FP = 1 } hero_mode;
typedef enum { HERO_MOD_QKV = 0, HERO_MOD_ATTN = 1, HERO_MOD_ATTN_OUT = 2, HERO_MOD_FC1 = 3, HERO_MOD_FC2 = 4 } hero_module;
typedef enum { HERO_PRESET_M1 = 1, HERO_PRESET_M2 = 2, HERO_PRESET_M3 = 3, HERO_PRESET_FP = 0 } hero_preset;

/* A matrix on the device.  data == NULL means "absent" wherever a tensor is optional.
 *   dtype : hero_dtype of the payload
 *   gran  : hero_gran; for HERO_I8 payloads says what `scale` holds:
 *           TWQ -> scale[rows], FWQ -> scale[cols], SQ -> scale[1], NONE -> no scale (value = code)
 *   scale : device float32; read for inputs and for FWQ/SQ outputs, WRITTEN for TWQ outputs. */
typedef struct {
  void* data;
  int32_t dtype;
  int32_t gran;
  int64_t rows;
  int64_t cols;
  int64_t ld;
  float* scale;
} hero_tensor;

typedef struct hero_handle hero_handle;

/* Create / destroy a handle on the current CUDA device.  Creation allocates the 4-byte device
 * error word and queries the device; it is the only place the library allocates. */
hero_status hero_create(hero_handle** out);
hero_status hero_destroy(hero_handle* h);
/* Text of the last error raised on the calling thread (never NULL). */
const char* hero_last_error(void);
/* Synchronize `stream`, read the device error word and clear it. */
hero_status hero_check(hero_handle* h, void* stream);
/* Number of kernels this handle has launched since creation (for benchmarks' accounting). */
int64_t hero_launch_count(const hero_handle* h);

/* ---------------------------------------------------------------------------------------------
 * LN^quant  (Sec. 2.2.1 Eq. 6-7 embedding flavour; Sec. 2.2.2 Eq. 19 and Sec. 2.2.3 Eq. 31
 * residual flavour).  One pass over each row:
 *     r[i,:]  = residual[i,:] + branch[i,:] + extra[i,:]        (each dequantized in fp32)
 *     y[i,:]  = (r - mean_i) / sqrt(biased_var_i + eps) * gamma + beta
 *     out     = TWQ: S[i] = absmax_j |y[i,j]| / 127 (zero row -> 1), q = clip(Round(y / S[i]))
 *               FWQ / SQ: q = clip(Round(y / S[j]))  with the given calibrated scale
 *               F16 / BF16: y rounded to that type
 *   residual : required.  I8 (TWQ / FWQ / SQ / NONE) or F16 / BF16, [M, H].
 *   branch   : optional second addend, I8 (FWQ / SQ / TWQ / NONE) or F16 / BF16 (X_o S_o of Eq. 19).
 *   extra    : optional third addend, F16 / BF16 (X_s of Eq. 7).
 *   token_ids != NULL selects the embedding gather of Eq. 7: `residual` is then the token table
 *       [V, H] I8 with TWQ scale [V], row ids[i]; `branch` the position table [P, H] F16/BF16, row
 *       (i mod seq_len); `extra` the sentence-type table [T, H], row type_ids[i].  M = n_tokens.
 *       P >= seq_len is required.  An id outside [0, V) or [0, T) is clamped to the nearest valid row and reported
 *       by the next hero_check() as HERO_ERR_INVALID_ARG.
 *   out      : I8 (gran TWQ: out.scale[M] is written; FWQ / SQ: out.scale is read) or F16 / BF16.
 *              out.data == NULL skips the normalisation (bare residual add into fp_out).
 *   fp_out   : optional F16 / BF16 copy of r (the FP residual stream of a pre-LN layer); when
 *              present the normalisation reads the stored (rounded) r.
 *   out_col_absmax : optional calibration observer (Sec. 2.1: FWQ / SQ scales come from calibration), device float[H]
 *              that the caller zeroes once: after the call entry j is max(old, max_i |t[i,j]|) of the FP tensor the
 *              call stores, t = out when out is F16 / BF16, t = fp_out when out.data is NULL.  The values observed are
 *              the stored (rounded) ones, so the result equals hero_absmax_observe on t bit for bit, without the
 *              second read.  An 8-bit out: HERO_ERR_UNSUPPORTED.
 * H must be a multiple of 16 and at most 16384.  M may be any size, including 0 (no launch).
 */
typedef struct {
  hero_tensor residual;
  hero_tensor branch;
  hero_tensor extra;
  const int32_t* token_ids; /* device [M] or NULL */
  const int32_t* type_ids;  /* device [M]; required with token_ids when extra is present */
  int32_t seq_len;
  int64_t n_tokens;         /* M for the gather flavour; ignored otherwise */
  const float* gamma;       /* device [H] */
  const float* beta;        /* device [H] */
  float eps;
  hero_tensor out;
  hero_tensor fp_out;
  float* out_col_absmax;    /* device [H] or NULL */
} hero_ln_args;

hero_status hero_layernorm_quant(hero_handle* h, const hero_ln_args* a, void* stream);

/* ---------------------------------------------------------------------------------------------
 * GeMM^quant with fused epilogue (Sec. 2.2.2 Eq. 14, 18, 20-23; Sec. 2.2.3 Eq. 28-30, 32).
 *     acc[i,j] = sum_k A[i,k] * W[j,k]                    exact INT32 (INT8 operands)
 *     v        = acc * rs[i] * w_scale[j] + bias[j]       rs = TWQ scale of A, or 1
 *     a        = act(v)                                   none | GELU(erf) | GELU(tanh)
 *     a       *= post_scale[j]                            (1 / S_a of GELU^quant; NULL = skip)
 *     out      = I8: clip(Round(a), -127, 127)            (Eq. 22: a bare Round once scales are folded)
 *                F16 / BF16: a rounded to that type
 *                I32: the raw accumulators (INT8 operands only; epilogue skipped; for verification)
 *   A    : [M, K] I8 (gran TWQ -> row scale applied; NONE / FWQ / SQ -> none: a feature-wise or
 *          static input scale must already be folded into W's rows, Eq. 23 / 32), or F16 / BF16
 *          for a module left in FP mode (then W has the same type and w_scale is ignored).
 *   W    : device [N][K], K contiguous, leading dimension ldw; same element type as A.  W is a constant of the model:
 *          kernels may fetch it before earlier work on the stream has completed, so it must not be written by work
 *          still in flight when the call is made (hero_quantize_weight takes care of this for its own outputs).
 *   out  : [M, N].  A TWQ output is refused (HERO_ERR_UNSUPPORTED): the paper keeps the row
 *          reduction out of GEMM epilogues (Sec. 2.1).
 *   out_col_absmax : device float[N] or NULL.  Calibration observer fused into the epilogue (Sec. 2.1: the static
 *          scales come from statistics of the un-quantized layer): out_col_absmax[j] = max(out_col_absmax[j],
 *          max_i |out[i][j]|) over the values as stored, the same statistic hero_absmax_observe takes from the finished
 *          tensor, without reading it again.  F16 / BF16 outputs only (HERO_ERR_UNSUPPORTED otherwise); accumulates, so
 *          zero it before the first calibration batch.
 * K must be a multiple of 16 bytes of elements and N a multiple of 16; M is arbitrary.
 */
typedef struct {
  hero_tensor A;
  const void* W;
  int64_t N;
  int64_t ldw;
  const float* w_scale;    /* device [N] (INT8 operands) */
  const float* bias;       /* device [N] or NULL */
  int32_t act;             /* hero_act */
  const float* post_scale; /* device [N] or NULL */
  hero_tensor out;
  float* out_col_absmax;   /* device [N] or NULL */
} hero_linear_args;

hero_status hero_w8a8_linear(hero_handle* h, const hero_linear_args* a, void* stream);

/* ---------------------------------------------------------------------------------------------
 * INT8 attention core (Sec. 2.2.2 Eq. 15-17).  Per (batch b, head h), rows of one sequence:
 *     A    = d~ (Q K^T),  d~ = s_q s_k / sqrt(dh)          INT32 -> fp32, never quantized
 *     P    = softmax(A) over the allowed keys              fully normalised
 *     P_u8 = clip(Round(P / s_p), 0, 255)                  unsigned ("asymmetric") INT8
 *     acc  = P_u8 V                                        exact INT32
 *     out  = I8: clip(Round(acc * s_p * s_v / out_scale[j]))  (FWQ [H]; SQ: one value)
 *            F16 / BF16: acc * s_p * s_v
 *   q, k, v : device pointers to element (0, 0) of [B*S, nh*dh] views with leading dimension ld
 *             (e.g. the three thirds of the QKV GEMM output, ld = 3H).  dtype I8, or F16 / BF16 for
 *             the FP attention of a module left in FP mode (then s_q, s_k, s_v, s_p are ignored and
 *             out = softmax(Q K^T / sqrt(dh)) V, quantized by out_scale when out is I8).
 *   mask    : HERO_MASK_NONE or HERO_MASK_CAUSAL; key_len (device int32 [B], optional) further
 *             limits the keys of sequence b to k < key_len[b].  A fully masked row outputs 0.
 *   dh is 64 or 128.
 */
/* How the INT8 core quantizes the softmax output.
 *   HERO_P_STATIC (the paper, Eq. 16): P_u8 = clip(Round(P / s_p)) of the normalised probabilities, s_p calibrated.
 *   HERO_P_ROWMAX (not in the paper; robust to long sequences, where probabilities below s_p / 2 vanish under the
 *     static scale): P~_u8 = Round(255 * exp(A - max_row A)), row sum l of the un-quantized exponentials in FP32,
 *     out = acc * s_v / (255 * l); s_p is ignored. */
typedef enum { HERO_P_STATIC = 0, HERO_P_ROWMAX = 1 } hero_p_mode;

typedef struct {
  const void* q;
  const void* k;
  const void* v;
  int32_t dtype;       /* hero_dtype of q, k, v */
  int64_t ld;
  int32_t B, S, nh, dh;
  float s_q, s_k, s_v, s_p;
  int32_t mask;        /* hero_mask */
  const int32_t* key_len;
  hero_tensor out;     /* [B*S, nh*dh]; I8 with gran FWQ (scale[H]) or SQ (scale[1]); or F16 / BF16 */
  float* p_absmax;     /* optional, F16 / BF16 core only: device float[1] holding a running maximum (the caller zeroes
                          it once); after the call it is max(old, largest softmax probability seen), from which
                          calibration takes s_p = p_absmax / 255 (Eq. 16).  NULL: not observed. */
  int32_t p_mode;      /* hero_p_mode: how P is quantized (INT8 core only); 0 = the paper's static scale */
  float* out_col_absmax; /* optional, F16 / BF16 core with an F16 / BF16 out only: device float[nh*dh] of running
                          per-column maxima of |out| as stored (the caller zeroes it once), equal bit for bit to
                          hero_absmax_observe on out; calibration takes the FWQ scale of X_attn from it (Eq. 17).
                          NULL: not observed.  Any other combination: HERO_ERR_UNSUPPORTED. */
} hero_attn_args;

hero_status hero_int8_attention(hero_handle* h, const hero_attn_args* a, void* stream);

/* The same core with its on-chip intermediates written out, for verification (Sec. 2.2.2 Eq. 15-17 name three
 * quantities that never leave the chip in hero_int8_attention: the INT32 result of Q K^T, the unsigned codes P_u8 and
 * the INT32 result of P_u8 V).  INT8 operands only, either p_mode; `a->out` is written as usual.  Slow (scalar stores):
 * for tests, not for the hot path.  Each pointer may be NULL.
 *   scores  : device int32 [B*nh][S][S]: scores[(b*nh + h)][i][k] = sum_c Q[i][c] K[k][c] (before the factor d~).
 *   p_codes : device uint8 [B*nh][S][S]: P_u8 of Eq. 16 (HERO_P_ROWMAX: P~_u8); a masked key inside a visited block holds 0.
 *             Both arrays are written for query row i at every key k < S of the 128-key blocks the kernel visits
 *             for that row (under a causal mask: blocks up to the one holding the diagonal); other entries are untouched.
 *   acc     : device int32 [B*S][nh*dh]: acc[i][j] = sum_k P_u8[i][k] V[k][j] of Eq. 17, before s_p s_v / S_attn;
 *             rows of a sequence without any allowed key are untouched. */
typedef struct {
  int32_t* scores;
  uint8_t* p_codes;
  int32_t* acc;
} hero_attn_probe;
hero_status hero_int8_attention_probe(hero_handle* h, const hero_attn_args* a, const hero_attn_probe* probe, void* stream);

/* ---------------------------------------------------------------------------------------------
 * One decode step of the INT8 attention core (Sec. 2.2.2 Eq. 15-17 for the single new token of each sequence of a
 * generative model; Sec. 1 names GPT-style models as targets) over an INT8 key / value cache.  Per (b, h), with
 * L = len[b] cache entries, the new token's own key and value included:
 *     A[k] = d~ (q . K[k]),  d~ = s_q s_k / sqrt(dh),  k < L;   P = softmax(A);   P_u8 = clip(Round(P / s_p), 0, 255)
 *     acc  = sum_k P_u8[k] V[k]   (exact INT32);   out = acc * s_p * s_v  ->  I8 by out.scale (FWQ [H] / SQ [1]) or F16 / BF16
 *   (HERO_P_ROWMAX: P~_u8 = Round(255 exp(A - max A)), out = acc * s_v / (255 * sum exp), s_p ignored): the row the
 *   causal prefill computes for the last of L tokens.
 *   q            : device I8 [B][nh*dh], row pitch ld_q elements
 *   k_cache, v_cache : device I8; entry t of sequence b starts at cache + b * batch_stride + t * ld_kv (elements), its
 *                  nh*dh features contiguous, head h at offset h*dh.  Pointers 16-byte aligned, ld_q / ld_kv /
 *                  batch_stride multiples of 16.  Read-only here unless k_new / v_new are given.
 *   k_new, v_new : optional device I8 [B][nh*dh] (row pitch ld_new): the new token's key and value, e.g. the other two
 *                  thirds of the QKV GeMM^quant output.  When given, entry len[b] - 1 of the caches is taken from them
 *                  and the call also stores them there (the append is fused); when NULL the caches already hold it.
 *   len          : device int32 [B]; 0 <= len[b] <= max_len; len[b] = 0 writes zeros for sequence b
 *   max_len      : host-side upper bound on len[b] (sizes the launch; a larger len[b] is treated as max_len); at most 98304
 *   out          : [B][nh*dh] I8 (gran FWQ scale[H] or SQ scale[1]) or F16 / BF16; dh is 64 or 128
 * Errors: HERO_ERR_INVALID_ARG / HERO_ERR_ALIGNMENT / HERO_ERR_UNSUPPORTED with hero_last_error() saying which.
 */
typedef struct {
  const void* q;
  int64_t ld_q;
  void* k_cache;
  void* v_cache;
  int64_t ld_kv;
  int64_t batch_stride;
  const void* k_new;
  const void* v_new;
  int64_t ld_new;
  const int32_t* len;
  int32_t max_len;
  int32_t B, nh, dh;
  float s_q, s_k, s_v, s_p;
  int32_t p_mode;      /* hero_p_mode */
  hero_tensor out;
} hero_decode_attn_args;

hero_status hero_int8_decode_attention(hero_handle* h, const hero_decode_attn_args* a, void* stream);

/* ---------------------------------------------------------------------------------------------
 * One transformer layer (Sec. 2.2.2-2.2.3, modes of Sec. 2.3 Table 1).
 * Post-LN (the paper's equations):  x_mid = LN1(x_in + Attn(x_in)); x_out = LN2(x_mid + MLP(x_mid)).
 * Pre-LN (GPT-shaped): h' = h + Attn(LN1(h [+ pending])); out = h' + MLP(LN2(h')) with the residual
 * stream h in fp_dtype.
 * A producer emits what its consumer's mode needs; an INT8 module contracts INT8 x INT8.
 */
typedef struct {
  const void* W;           /* device [N][K]: I8 when the module is INT8, else fp_dtype */
  const float* w_scale;    /* device [N]; INT8 modules */
  const float* bias;       /* device [N] or NULL */
  const float* post_scale; /* device [N] or NULL: multiplies after the activation (1/S_a; 1/S_q.. for an
                              FP QKV feeding INT8 attention) */
} hero_linear_params;

typedef struct {
  int32_t arch;            /* hero_arch */
  int32_t B, S, H, nh, F;
  int32_t act;             /* hero_act of the MLP */
  float eps;
  int32_t mask;            /* hero_mask */
  int32_t fp_dtype;        /* HERO_F16 or HERO_BF16: type of every FP tensor at a module border */
  int32_t mode[5];         /* hero_mode per hero_module */
  int32_t gran_in;         /* granularity of the INT8 tensor feeding QKV (TWQ | FWQ | SQ) */
  int32_t gran_mid;        /* granularity of the INT8 tensor feeding FC1 */
  int32_t gran_attn;       /* granularity of X_attn (FWQ | SQ) */
  int32_t gran_out;        /* post-LN layer output: TWQ | FWQ | SQ, or NONE for an FP output */
  const float* s_in;       /* device: FWQ [H] / SQ [1] scale of the tensor feeding QKV (pre-LN: LN1 output) */
  const float* s_mid;      /* device: same for the tensor feeding FC1 */
  const float* s_attn;     /* device: FWQ [H] / SQ [1] scale of X_attn */
  const float* s_o;        /* device [H]: FWQ scale X_o stands for (folded into W_o; used by LN) */
  const float* s_x2;       /* device [H]: FWQ scale X_2 stands for */
  const float* s_out;      /* device: FWQ [H] / SQ [1] scale of a non-TWQ INT8 layer output */
  float s_q, s_k, s_v, s_p;
  hero_linear_params qkv, o, fc1, fc2;
  const float* ln1_g; const float* ln1_b;
  const float* ln2_g; const float* ln2_b;
  int32_t p_mode;          /* hero_p_mode of the INT8 attention core (0 = the paper's static S_p) */
  int32_t payload;         /* 8-bit type of the modules in HERO_MODE_INT8: HERO_I8 (0, the paper) or HERO_F8, the FP8
                              variant: every 8-bit tensor at a module border, the weights (W of those modules holds
                              e4m3 bytes) and P are e4m3, every scale is absmax / 448, the contractions accumulate in
                              FP32.  With HERO_F8: p_mode must be static, `in` (post-LN) and an 8-bit `out` are HERO_F8,
                              and an FP attention core cannot feed an 8-bit attention-output linear
                              (HERO_ERR_UNSUPPORTED). */
} hero_layer_desc;

/* ---------------------------------------------------------------------------------------------
 * Calibration on the device (Sec. 2.1: the static scales of Eq. 4-5 come from statistics of the un-quantized
 * layer over calibration data; Eq. 2 and Eq. 20-23 / 32 for the weights).  Run the layer's modules in FP mode
 * through the entry points above and observe every tensor at an operator border with hero_absmax_observe
 * (the softmax probabilities through hero_attn_args.p_absmax); a scale is absmax / 127 (absmax / 255 for P),
 * 1 when the statistic is 0.
 *
 * hero_absmax_observe: running absolute maxima of x ([rows, cols] F16 / BF16, cols and ld multiples of 8).
 *   col_absmax    : device float[cols] or NULL: col_absmax[j] = max(col_absmax[j], max_i |x[i][j]|)   (Eq. 4)
 *   tensor_absmax : device float[1]    or NULL: max(old, max_ij |x[i][j]|)                            (Eq. 5)
 *   Both accumulate, so several calibration batches can be observed one after another; zero them first.
 *
 * hero_quantize_weight: fold, then column-wise symmetric INT8 (Eq. 2 after Eq. 20-23 / 32), for W [N][K] FP32
 * (row n = output feature n; K, ldw, ldq multiples of 4):
 *     W~[n][k] = W[n][k] * in_scale[k] / out_scale[n]      in_scale [K] or NULL (the consumer-side fold of the
 *                                                          input's FWQ / SQ scale), out_scale [N] or NULL (the
 *                                                          producer-side fold of the output's scale)
 *     w_scale[n] = max_k |W~[n][k]| / 127  (1 if the row is zero);   Wq[n][k] = clip(Round(W~[n][k] / w_scale[n]))
 *     bias_out[n] = bias[n] / out_scale[n]                 when bias_out is given (bias NULL reads as 0)
 *   All pointers are device pointers; outputs are caller-owned.  The paper gives the equations, not an interface. */
hero_status hero_absmax_observe(hero_handle* h, const hero_tensor* x, float* col_absmax, float* tensor_absmax,
                                void* stream);
/* Percentile clipping of a static scale (the truncation threshold the paper leaves un-tuned, Sec. 3): adds the
 * histogram of |x| over HERO_HIST_BINS equal bins of [0, bound) to hist (device uint64[HERO_HIST_BINS], accumulating;
 * values >= bound fall into the last bin).  With bound = the tensor's absmax, the q-th percentile is the upper edge
 * of the first bin at which the cumulative count reaches q of the total. */
#define HERO_HIST_BINS 2048
hero_status hero_abs_histogram(hero_handle* h, const hero_tensor* x, float bound, uint64_t* hist, void* stream);
hero_status hero_quantize_weight(hero_handle* h, const float* W, int64_t ldw, int32_t N, int32_t K,
                                 const float* in_scale, const float* out_scale, const float* bias, int8_t* Wq,
                                 int64_t ldq, float* w_scale, float* bias_out, void* stream);

/* The same fold for the FP8 variant of the method (Sec. 2.1: the approach "carries over to FP8"): the payload is e4m3,
 * w_scale[n] = max_k |W~[n][k]| / 448 (1 if the row is zero) and Wq[n][k] is the byte of the saturating
 * round-to-nearest-even conversion of W~[n][k] / w_scale[n].  Arguments as hero_quantize_weight. */
hero_status hero_quantize_weight_f8(hero_handle* h, const float* W, int64_t ldw, int32_t N, int32_t K,
                                    const float* in_scale, const float* out_scale, const float* bias, uint8_t* Wq,
                                    int64_t ldq, float* w_scale, float* bias_out, void* stream);

/* Fill desc->mode from a Table 1 preset (M1, M2, M3) or all-FP. */
hero_status hero_mode_preset(int32_t preset, int32_t mode_out[5]);
/* Scratch the layer needs for M tokens. */
hero_status hero_layer_workspace_bytes(const hero_layer_desc* d, int64_t M, size_t* bytes);
/* Where hero_layer_forward leaves the tensors at the operator borders (Sec. 2.2.2-2.2.3) inside the workspace: byte
 * offsets from the workspace pointer, valid after a forward call has completed, for inspection and stage-by-stage
 * checking.  Every tensor is row-major [M, cols] with ld = cols, INT8 or fp_dtype as the module modes dictate.
 *   qkv [M,3H], x_attn [M,H], x_o [M,H], x_mid [M,H] (+ x_mid_scale [M] FP32 when gran_mid is TWQ), a [M,F] (the
 *   GELU^quant output), x_2 [M,H]; pre-LN only: x_in [M,H] (+ x_in_scale [M]), h_in and h_mid [M,H] in fp_dtype
 *   (h_in holds h + pending when a pending branch was given).  Offsets that do not apply are 0. */
typedef struct hero_layer_layout {
  size_t qkv, x_attn, x_o, x_mid, x_mid_scale, a, x_2, x_in, x_in_scale, h_in, h_mid;
  size_t total;            /* = hero_layer_workspace_bytes */
} hero_layer_layout;
hero_status hero_layer_workspace_layout(const hero_layer_desc* d, int64_t M, hero_layer_layout* layout);
/*   in      : post-LN: X_in [M, H] I8 (+scale per gran_in) or fp_dtype when QKV is FP.
 *             pre-LN : residual stream h [M, H] in fp_dtype.
 *   pending : pre-LN only, optional: a branch (I8 FWQ or fp_dtype) still to be added to h, i.e. the
 *             previous layer's X_2; the add is fused into LN1's kernel.
 *   out     : post-LN: X_out (I8 TWQ -> out.scale[M] written; I8 FWQ/SQ; or fp_dtype).
 *             pre-LN : h_out = h' + X_2 in fp_dtype (the closing add of a lone layer).
 *   workspace: device scratch of at least hero_layer_workspace_bytes(), 256-byte aligned. */
hero_status hero_layer_forward(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in,
                               const hero_tensor* pending, const hero_tensor* out, void* workspace,
                               size_t workspace_bytes, void* stream);

/* One decode step of the layer: the new token of each of the B sequences (in: [B, H], typed as for hero_layer_forward)
 * goes through the same modules, the attention core in its decode form (hero_int8_decode_attention) against this
 * layer's INT8 key / value cache.  The step stores the new token's key and value at entry len[b] - 1 of the caches
 * (the caller increments len before the call and owns the caches) and writes out: [B, H].  The attention module must
 * be HERO_MODE_INT8 with the INT8 payload; desc->S is not used; the workspace is the one of a forward pass or at least
 * hero_layer_workspace_bytes(desc, B).  The result equals row len[b] - 1 of a causal forward pass over the sequence
 * so far (up to rounding ties). */
typedef struct {
  void* k_cache;           /* device I8, entry t of sequence b at k_cache + b * batch_stride + t * ld_kv, H features */
  void* v_cache;
  int64_t ld_kv;
  int64_t batch_stride;
  const int32_t* len;      /* device int32 [B]: cache entries including the new token */
  int32_t max_len;         /* host-side upper bound on len[b] */
} hero_kv_cache;

hero_status hero_layer_decode(hero_handle* h, const hero_layer_desc* desc, const hero_kv_cache* kv, const hero_tensor* in,
                              const hero_tensor* pending, const hero_tensor* out, void* workspace, size_t workspace_bytes,
                              void* stream);

/* The same layer (Sec. 2.2.2-2.2.3) called with HOST activation buffers: copies `in_host` (payload and, for
 * a token-wise input, its per-row scales) into the caller's device staging tensor `in_dev`, runs
 * hero_layer_forward, copies the result back into `out_host` and synchronizes the stream.  Host buffers
 * should be page-locked for the copies to be asynchronous.  Weights, calibrated scales, staging tensors and
 * workspace stay device-resident and caller-owned; nothing is allocated. */
hero_status hero_layer_forward_host(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in_host,
                                    const hero_tensor* out_host, const hero_tensor* in_dev, const hero_tensor* out_dev,
                                    void* workspace, size_t workspace_bytes, void* stream);
/* The same without the final synchronisation: the copies and the layer are only enqueued on `stream`, and `out_host`
 * is valid once the caller has synchronised that stream.  Several calls on different streams, each with its own
 * staging tensors, workspace and host output buffer, overlap one step's copies with another step's kernels. */
hero_status hero_layer_forward_host_async(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in_host,
                                          const hero_tensor* out_host, const hero_tensor* in_dev,
                                          const hero_tensor* out_dev, void* workspace, size_t workspace_bytes, void* stream);

/* A stack of layers (the paper's models are stacks of the layer of Sec. 2.2.2-2.2.3 behind the embedding LN^quant of
 * Sec. 2.2.1): host-side sequencing only, one hero_layer_forward per layer on `stream`, layer i reading edges[i] and
 * writing edges[i + 1], all layers sharing one workspace (at least the largest hero_layer_workspace_bytes among them).
 *   layers   : host array [n_layers] of layer descriptors
 *   edges    : host array [n_layers + 1] of DEVICE tensors, typed as each layer's `in` / `out` (hero_layer_forward)
 *   pending  : host array [n_layers] or NULL: pre-LN only, the branch still to be added to layer i's input
 *   entry_in : optional DEVICE tensor [M, H] F16 / BF16; when present the entry LN^quant (plain flavour of Eq. 6-7,
 *              entry_gamma / entry_beta / entry_eps) turns it into edges[0] before layer 0 runs. */
typedef struct {
  int32_t n_layers;
  const hero_layer_desc* layers;
  const hero_tensor* edges;
  const hero_tensor* pending;
  hero_tensor entry_in;
  const float* entry_gamma;
  const float* entry_beta;
  float entry_eps;
} hero_stack_desc;
hero_status hero_stack_forward(hero_handle* h, const hero_stack_desc* stack, void* workspace, size_t workspace_bytes,
                               void* stream);
/* The same with HOST activation buffers, enqueued on `stream` without a final synchronisation: in_host is copied into
 * entry_in (when the stack has an entry LN^quant) or into edges[0] (payload and, for a token-wise tensor, its row
 * scales), the stack runs, and edges[n_layers] is copied into out_host, which is valid once the caller has
 * synchronised the stream.  Host buffers should be page-locked.  Nothing is allocated. */
hero_status hero_stack_forward_host_async(hero_handle* h, const hero_stack_desc* stack, const hero_tensor* in_host,
                                          const hero_tensor* out_host, void* workspace, size_t workspace_bytes, void* stream);

/* The layer forward for callers that cannot allocate device memory (the paper has no counterpart: it describes
 * no software interface).  Who needs it: code that runs inside another framework's fixed memory plan, real-time
 * or plugin paths where an allocation might block or fail late, processes that own only the buffers they were
 * started with.  It takes no handle and no workspace and calls no cudaMalloc / cudaFree or any other allocating
 * routine: its scratch is a 64 MiB array built into the library image, present on every GPU that loads the
 * library until the process exits.
 *   - A layer whose workspace (hero_layer_workspace_bytes) exceeds 64 MiB is refused with HERO_ERR_WORKSPACE.
 *   - The first call on a device looks up the array's device address and the driver's tensor-map encoder; make
 *     that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call left in it (nothing in it
 *     needs clearing: each call overwrites what it reads).  Two calls that overlap on the GPU, e.g. on two
 *     streams, race on it: serialize them.
 *   - Host threads may call it concurrently as far as the host side goes, but their kernels share the one array:
 *     unless the caller serializes them on the GPU (one stream, or events between streams) they race on it.
 *   - A bounded device-side wait that gives up is recorded in a device word of the library image (there is no
 *     handle for hero_check to look at); hero_static_check reads it.
 * Inputs, outputs, weights and scales are passed exactly as for hero_layer_forward. */
hero_status hero_layer_forward_static(const hero_layer_desc* d, const hero_tensor* in, const hero_tensor* pending,
                                      const hero_tensor* out, void* stream);
/* hero_check for hero_layer_forward_static (the paper has no counterpart either): synchronizes `stream`, reads the
 * device error word of the current device, clears it, and returns HERO_OK or HERO_ERR_DEVICE_TIMEOUT.  Allocates
 * nothing (a symbol copy). */
hero_status hero_static_check(void* stream);

/* Per-launch device timing for benchmarks (no counterpart in the paper, which measured nothing): between
 * _begin and _end every kernel the handle launches is bracketed by a pair of CUDA events on its stream.
 * _end waits for them and returns, per launch in order, the elapsed milliseconds and the kernel family
 * (1 = LN^quant, 2 = GeMM^quant, 3 = attention core).  Arrays must hold max_launches entries. */
hero_status hero_profile_begin(hero_handle* h, int32_t max_launches);
hero_status hero_profile_end(hero_handle* h, float* ms_out, int32_t* tag_out, int32_t* n_out);

#ifdef __cplusplus
}
#endif
#endif /* HERO_H_ */
