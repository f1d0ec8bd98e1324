// hero_layer_forward: one transformer layer (Sec. 2.2.2-2.2.3) under the per-module modes of Table 1.
// Host-side sequencing only: seven kernel launches on one stream (QKV GeMM^quant, attention core,
// attention-output GeMM^quant, LN^quant, FC1 + GELU^quant, FC2 GeMM^quant, LN^quant), every
// intermediate in the caller's workspace.  No standalone quantize kernel exists: each tensor is
// quantized by the epilogue of its producer, and a producer emits what its consumer's mode needs.
#include "common.cuh"

namespace hero {

struct LayerPlan {
  size_t off_qkv, off_attn, off_o, off_mid, off_mid_scale, off_a, off_x2, off_xin, off_xin_scale, off_hin, off_hmid;
  size_t total;
};

static inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

static hero_status plan_layer(const hero_layer_desc* d, int64_t M, LayerPlan* pl) {
  HERO_REQUIRE(d != nullptr, HERO_ERR_INVALID_ARG, "layer descriptor is NULL");
  HERO_REQUIRE(d->arch == HERO_POST_LN || d->arch == HERO_PRE_LN, HERO_ERR_INVALID_ARG, "unknown arch %d", d->arch);
  HERO_REQUIRE(d->B > 0 && d->S > 0 && d->H > 0 && d->nh > 0 && d->F > 0 && d->H % d->nh == 0, HERO_ERR_INVALID_ARG,
               "bad layer dimensions");
  HERO_REQUIRE(M == (int64_t)d->B * d->S || M == (int64_t)d->B, HERO_ERR_INVALID_ARG, "M=%lld is neither B*S (a forward pass) nor B (a decode step)",
               (long long)M);
  HERO_REQUIRE(is_fp16ish(d->fp_dtype), HERO_ERR_INVALID_ARG, "fp_dtype must be F16 or BF16");
  for (int i = 0; i < 5; ++i)
    HERO_REQUIRE(d->mode[i] == HERO_MODE_INT8 || d->mode[i] == HERO_MODE_FP, HERO_ERR_INVALID_ARG, "mode[%d]=%d", i, d->mode[i]);
  const size_t H = d->H, F = d->F, m = (size_t)M;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
  pl->off_qkv = take(m * 3 * H * 2);
  pl->off_attn = take(m * H * 2);
  pl->off_o = take(m * H * 2);
  pl->off_mid = take(m * H * 2);
  pl->off_mid_scale = take(m * 4);
  pl->off_a = take(m * F * 2);
  pl->off_x2 = take(m * H * 2);
  pl->off_xin = pl->off_xin_scale = pl->off_hin = pl->off_hmid = 0;
  if (d->arch == HERO_PRE_LN) {
    pl->off_xin = take(m * H * 2);
    pl->off_xin_scale = take(m * 4);
    pl->off_hin = take(m * H * 2);
    pl->off_hmid = take(m * H * 2);
  }
  pl->total = o;
  return HERO_OK;
}

static hero_tensor mk(void* data, int dtype, int gran, int64_t rows, int64_t cols, const float* scale) {
  hero_tensor t;
  t.data = data; t.dtype = dtype; t.gran = gran; t.rows = rows; t.cols = cols; t.ld = cols;
  t.scale = const_cast<float*>(scale);
  return t;
}
static hero_tensor none() { return mk(nullptr, 0, 0, 0, 0, nullptr); }

}  // namespace hero

extern "C" hero_status hero_layer_workspace_bytes(const hero_layer_desc* d, int64_t M, size_t* bytes) {
  using namespace hero;
  HERO_REQUIRE(bytes != nullptr, HERO_ERR_INVALID_ARG, "bytes is NULL");
  LayerPlan pl;
  hero_status st = plan_layer(d, M, &pl);
  if (st != HERO_OK) return st;
  *bytes = pl.total;
  return HERO_OK;
}

extern "C" hero_status hero_layer_workspace_layout(const hero_layer_desc* d, int64_t M, hero_layer_layout* layout) {
  using namespace hero;
  HERO_REQUIRE(layout != nullptr, HERO_ERR_INVALID_ARG, "layout is NULL");
  LayerPlan pl;
  hero_status st = plan_layer(d, M, &pl);
  if (st != HERO_OK) return st;
  layout->qkv = pl.off_qkv; layout->x_attn = pl.off_attn; layout->x_o = pl.off_o; layout->x_mid = pl.off_mid;
  layout->x_mid_scale = pl.off_mid_scale; layout->a = pl.off_a; layout->x_2 = pl.off_x2; layout->x_in = pl.off_xin;
  layout->x_in_scale = pl.off_xin_scale; layout->h_in = pl.off_hin; layout->h_mid = pl.off_hmid;
  layout->total = pl.total;
  return HERO_OK;
}

namespace hero {
// The layer on M = B*S tokens (kv == NULL), or one decode step on M = B new tokens against the layer's key / value
// cache: the same launches with the attention core replaced by its decode form.
static hero_status layer_impl(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in, const hero_tensor* pending,
                              const hero_tensor* out, void* workspace, size_t workspace_bytes, void* stream,
                              const hero_kv_cache* kv) {
  HERO_REQUIRE(h && d && in && out, HERO_ERR_INVALID_ARG, "hero_layer_forward: NULL argument");
  const int64_t M = in->rows;
  HERO_REQUIRE(M == (kv ? (int64_t)d->B : (int64_t)d->B * d->S), HERO_ERR_INVALID_ARG, "in has %lld rows: %s expected", (long long)M,
               kv ? "B (one new token per sequence)" : "B*S");
  LayerPlan pl;
  hero_status st = plan_layer(d, M, &pl);
  if (st != HERO_OK) return st;
  HERO_REQUIRE(workspace != nullptr && (reinterpret_cast<uintptr_t>(workspace) & 255) == 0, HERO_ERR_ALIGNMENT,
               "workspace must be a 256-byte aligned device pointer");
  HERO_REQUIRE(workspace_bytes >= pl.total, HERO_ERR_WORKSPACE, "workspace too small: %zu < %zu", workspace_bytes, pl.total);
  HERO_REQUIRE(in->cols == d->H && out->rows == M && out->cols == d->H, HERO_ERR_INVALID_ARG, "in / out shape mismatch");
  const bool pre = d->arch == HERO_PRE_LN;
  HERO_REQUIRE(pre || pending == nullptr || pending->data == nullptr, HERO_ERR_INVALID_ARG, "pending is for pre-LN layers only");

  const int H = d->H, F = d->F, fp = d->fp_dtype;
  HERO_REQUIRE(d->payload == HERO_I8 || d->payload == HERO_F8, HERO_ERR_INVALID_ARG, "payload %d: HERO_I8 or HERO_F8 expected", d->payload);
  const int q8 = d->payload;   // the 8-bit type at every border of the modules in 8-bit mode
  const bool qkv8 = d->mode[HERO_MOD_QKV] == HERO_MODE_INT8, attn8 = d->mode[HERO_MOD_ATTN] == HERO_MODE_INT8;
  const bool o8 = d->mode[HERO_MOD_ATTN_OUT] == HERO_MODE_INT8, fc18 = d->mode[HERO_MOD_FC1] == HERO_MODE_INT8;
  const bool fc28 = d->mode[HERO_MOD_FC2] == HERO_MODE_INT8;
  uint8_t* ws = static_cast<uint8_t*>(workspace);

  // the INT8 tensor an LN emits for an INT8 consumer, by granularity (Eq. 3-5)
  auto ln_out = [&](void* data, bool int8, int gran, const float* static_scale, float* twq_scale) -> hero_tensor {
    if (!int8) return mk(data, fp, HERO_GRAN_NONE, M, H, nullptr);
    if (gran == HERO_GRAN_TWQ) return mk(data, q8, HERO_GRAN_TWQ, M, H, twq_scale);
    return mk(data, q8, gran, M, H, static_scale);
  };
  HERO_REQUIRE(d->gran_in == HERO_GRAN_TWQ || d->gran_in == HERO_GRAN_FWQ || d->gran_in == HERO_GRAN_SQ, HERO_ERR_INVALID_ARG, "gran_in");
  HERO_REQUIRE(d->gran_mid == HERO_GRAN_TWQ || d->gran_mid == HERO_GRAN_FWQ || d->gran_mid == HERO_GRAN_SQ, HERO_ERR_INVALID_ARG, "gran_mid");
  HERO_REQUIRE(d->gran_attn == HERO_GRAN_FWQ || d->gran_attn == HERO_GRAN_SQ, HERO_ERR_UNSUPPORTED,
               "X_attn is feature-wise or static (a GEMM-like epilogue cannot reduce over a row, Sec. 2.1)");

  hero_tensor x_in = *in;       // what feeds QKV
  hero_tensor h_cur = *in;      // pre-LN: the FP residual stream
  if (pre) {
    HERO_REQUIRE(is_fp16ish(in->dtype) && in->dtype == fp, HERO_ERR_INVALID_ARG, "pre-LN: `in` is the residual stream in fp_dtype");
    hero_ln_args a;
    memset(&a, 0, sizeof(a));
    a.residual = *in;
    const bool has_pending = pending && pending->data;
    if (has_pending) a.branch = *pending;
    a.gamma = d->ln1_g; a.beta = d->ln1_b; a.eps = d->eps;
    a.out = ln_out(ws + pl.off_xin, qkv8, d->gran_in, d->s_in, reinterpret_cast<float*>(ws + pl.off_xin_scale));
    if (has_pending) {
      a.fp_out = mk(ws + pl.off_hin, fp, HERO_GRAN_NONE, M, H, nullptr);
      h_cur = a.fp_out;
    }
    if ((st = hero_layernorm_quant(h, &a, stream)) != HERO_OK) return st;
    x_in = a.out;
  } else {
    HERO_REQUIRE(qkv8 ? in->dtype == q8 : in->dtype == fp, HERO_ERR_INVALID_ARG,
                 "post-LN: `in` must have the layer's 8-bit payload when the QKV module is 8-bit, else fp_dtype");
  }

  // ---- QKV GeMM^quant (Eq. 14, 20-22)
  if (q8 == HERO_F8) {
    HERO_REQUIRE(!attn8 || d->p_mode == HERO_P_STATIC, HERO_ERR_UNSUPPORTED, "the e4m3 attention core has the static P quantizer only");
    HERO_REQUIRE(attn8 || !o8, HERO_ERR_UNSUPPORTED, "e4m3 payload: an FP attention core cannot feed an 8-bit attention-output linear");
  }
  const int qkv_dt = attn8 ? q8 : fp;
  const size_t qkv_es = dtype_size(qkv_dt);
  hero_tensor qkv = mk(ws + pl.off_qkv, qkv_dt, HERO_GRAN_NONE, M, 3 * H, nullptr);
  {
    hero_linear_args a;
    memset(&a, 0, sizeof(a));
    a.A = x_in; a.W = d->qkv.W; a.N = 3 * H; a.ldw = H;
    a.w_scale = d->qkv.w_scale; a.bias = d->qkv.bias; a.act = HERO_ACT_NONE; a.post_scale = d->qkv.post_scale;
    a.out = qkv;
    if ((st = hero_w8a8_linear(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- attention core (Eq. 15-17)
  hero_tensor x_attn = o8 ? mk(ws + pl.off_attn, q8, d->gran_attn, M, H, d->s_attn)
                          : mk(ws + pl.off_attn, fp, HERO_GRAN_NONE, M, H, nullptr);
  if (kv) {
    // decode: the query and the new key / value are the thirds of the QKV rows; the step appends them to the cache
    HERO_REQUIRE(attn8 && q8 == HERO_I8, HERO_ERR_UNSUPPORTED, "a decode step needs the INT8 attention core");
    hero_decode_attn_args a;
    memset(&a, 0, sizeof(a));
    const int8_t* base = static_cast<const int8_t*>(qkv.data);
    a.q = base; a.ld_q = 3 * H;
    a.k_new = base + H; a.v_new = base + 2 * H; a.ld_new = 3 * H;
    a.k_cache = kv->k_cache; a.v_cache = kv->v_cache; a.ld_kv = kv->ld_kv; a.batch_stride = kv->batch_stride;
    a.len = kv->len; a.max_len = kv->max_len;
    a.B = d->B; a.nh = d->nh; a.dh = H / d->nh;
    a.s_q = d->s_q; a.s_k = d->s_k; a.s_v = d->s_v; a.s_p = d->s_p;
    a.p_mode = d->p_mode;
    a.out = x_attn;
    if ((st = hero_int8_decode_attention(h, &a, stream)) != HERO_OK) return st;
  } else {
    hero_attn_args a;
    memset(&a, 0, sizeof(a));
    uint8_t* base = static_cast<uint8_t*>(qkv.data);
    a.q = base; a.k = base + (size_t)H * qkv_es; a.v = base + (size_t)2 * H * qkv_es;
    a.dtype = qkv_dt; a.ld = 3 * H;
    a.B = d->B; a.S = d->S; a.nh = d->nh; a.dh = H / d->nh;
    a.s_q = d->s_q; a.s_k = d->s_k; a.s_v = d->s_v; a.s_p = d->s_p;
    a.mask = d->mask; a.key_len = nullptr;
    a.p_mode = d->p_mode;
    a.out = x_attn;
    if ((st = hero_int8_attention(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- attention-output GeMM^quant (Eq. 18, 23): the FWQ / SQ scale of X_attn lives in W~_o's rows
  hero_tensor x_o = o8 ? mk(ws + pl.off_o, q8, HERO_GRAN_FWQ, M, H, d->s_o) : mk(ws + pl.off_o, fp, HERO_GRAN_NONE, M, H, nullptr);
  {
    hero_linear_args a;
    memset(&a, 0, sizeof(a));
    a.A = x_attn; a.A.gran = HERO_GRAN_NONE; a.A.scale = nullptr;
    a.W = d->o.W; a.N = H; a.ldw = H;
    a.w_scale = d->o.w_scale; a.bias = d->o.bias; a.act = HERO_ACT_NONE; a.post_scale = d->o.post_scale;
    a.out = x_o; a.out.gran = HERO_GRAN_NONE; a.out.scale = nullptr;
    if ((st = hero_w8a8_linear(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- LN^quant (Eq. 19): residual + attention branch -> the tensor feeding FC1
  hero_tensor x_mid = ln_out(ws + pl.off_mid, fc18, d->gran_mid, d->s_mid, reinterpret_cast<float*>(ws + pl.off_mid_scale));
  hero_tensor h_mid = none();
  {
    hero_ln_args a;
    memset(&a, 0, sizeof(a));
    a.residual = pre ? h_cur : *in;
    a.branch = x_o;
    a.gamma = pre ? d->ln2_g : d->ln1_g; a.beta = pre ? d->ln2_b : d->ln1_b; a.eps = d->eps;
    a.out = x_mid;
    if (pre) { h_mid = mk(ws + pl.off_hmid, fp, HERO_GRAN_NONE, M, H, nullptr); a.fp_out = h_mid; }
    if ((st = hero_layernorm_quant(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- FC1 + GELU^quant (Eq. 28-29): X_1 never leaves the epilogue's registers
  hero_tensor act = fc28 ? mk(ws + pl.off_a, q8, HERO_GRAN_NONE, M, F, nullptr) : mk(ws + pl.off_a, fp, HERO_GRAN_NONE, M, F, nullptr);
  {
    hero_linear_args a;
    memset(&a, 0, sizeof(a));
    a.A = x_mid; a.W = d->fc1.W; a.N = F; a.ldw = H;
    a.w_scale = d->fc1.w_scale; a.bias = d->fc1.bias; a.act = d->act; a.post_scale = d->fc1.post_scale;
    a.out = act;
    if ((st = hero_w8a8_linear(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- FC2 GeMM^quant (Eq. 30, 32)
  hero_tensor x_2 = fc28 ? mk(ws + pl.off_x2, q8, HERO_GRAN_FWQ, M, H, d->s_x2) : mk(ws + pl.off_x2, fp, HERO_GRAN_NONE, M, H, nullptr);
  {
    hero_linear_args a;
    memset(&a, 0, sizeof(a));
    a.A = act; a.W = d->fc2.W; a.N = H; a.ldw = F;
    a.w_scale = d->fc2.w_scale; a.bias = d->fc2.bias; a.act = HERO_ACT_NONE; a.post_scale = d->fc2.post_scale;
    a.out = x_2; a.out.gran = HERO_GRAN_NONE; a.out.scale = nullptr;
    if ((st = hero_w8a8_linear(h, &a, stream)) != HERO_OK) return st;
  }
  // ---- LN^quant (Eq. 31) / closing residual add of a pre-LN layer
  {
    hero_ln_args a;
    memset(&a, 0, sizeof(a));
    a.branch = x_2;
    if (pre) {
      HERO_REQUIRE(out->dtype == fp, HERO_ERR_INVALID_ARG, "pre-LN: out is the residual stream in fp_dtype");
      a.residual = h_mid;
      a.fp_out = *out;
    } else {
      a.residual = x_mid;
      a.gamma = d->ln2_g; a.beta = d->ln2_b; a.eps = d->eps;
      a.out = *out;
      if (is_q8(out->dtype) && out->gran != HERO_GRAN_TWQ && out->scale == nullptr) a.out.scale = const_cast<float*>(d->s_out);
    }
    if ((st = hero_layernorm_quant(h, &a, stream)) != HERO_OK) return st;
  }
  return HERO_OK;
}
}  // namespace hero

extern "C" hero_status hero_layer_forward(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in,
                                          const hero_tensor* pending, const hero_tensor* out, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  return hero::layer_impl(h, d, in, pending, out, workspace, workspace_bytes, stream, nullptr);
}

extern "C" hero_status hero_layer_decode(hero_handle* h, const hero_layer_desc* d, const hero_kv_cache* kv, const hero_tensor* in,
                                         const hero_tensor* pending, const hero_tensor* out, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  using namespace hero;
  HERO_REQUIRE(kv && kv->k_cache && kv->v_cache && kv->len, HERO_ERR_INVALID_ARG, "hero_layer_decode: the key / value cache is required");
  return layer_impl(h, d, in, pending, out, workspace, workspace_bytes, stream, kv);
}

extern "C" hero_status hero_layer_forward_host_async(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in_host,
                                                     const hero_tensor* out_host, const hero_tensor* in_dev,
                                                     const hero_tensor* out_dev, void* workspace, size_t workspace_bytes,
                                                     void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && d && in_host && out_host && in_dev && out_dev, HERO_ERR_INVALID_ARG, "hero_layer_forward_host: NULL argument");
  HERO_REQUIRE(in_host->dtype == in_dev->dtype && in_host->rows == in_dev->rows && in_host->cols == in_dev->cols &&
               out_host->dtype == out_dev->dtype && out_host->rows == out_dev->rows && out_host->cols == out_dev->cols,
               HERO_ERR_INVALID_ARG, "host and device staging tensors must agree in type and shape");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t ies = dtype_size(in_dev->dtype), oes = dtype_size(out_dev->dtype);
  HERO_REQUIRE(ies && oes, HERO_ERR_INVALID_ARG, "unknown dtype");
  auto scale_len = [](const hero_tensor& t) -> size_t {
    if (!is_q8(t.dtype)) return 0;
    return t.gran == HERO_GRAN_TWQ ? (size_t)t.rows : 0;   // calibrated FWQ / SQ scales already live on the device
  };
  // host -> device: the activation payload and, for a token-wise input, its per-row scales
  // contiguous on both sides: one linear copy (the pitched form is kept for strided views)
  if (in_dev->ld == in_dev->cols && in_host->ld == in_host->cols)
    HERO_CUDA(cudaMemcpyAsync(in_dev->data, in_host->data, (size_t)in_dev->rows * in_dev->cols * ies, cudaMemcpyHostToDevice, s));
  else
    HERO_CUDA(cudaMemcpy2DAsync(in_dev->data, in_dev->ld * ies, in_host->data, in_host->ld * ies, in_dev->cols * ies,
                                in_dev->rows, cudaMemcpyHostToDevice, s));
  if (scale_len(*in_dev))
    HERO_CUDA(cudaMemcpyAsync(in_dev->scale, in_host->scale, scale_len(*in_dev) * sizeof(float), cudaMemcpyHostToDevice, s));
  hero_status st = hero_layer_forward(h, d, in_dev, nullptr, out_dev, workspace, workspace_bytes, stream);
  if (st != HERO_OK) return st;
  if (out_dev->ld == out_dev->cols && out_host->ld == out_host->cols)
    HERO_CUDA(cudaMemcpyAsync(out_host->data, out_dev->data, (size_t)out_dev->rows * out_dev->cols * oes, cudaMemcpyDeviceToHost, s));
  else
    HERO_CUDA(cudaMemcpy2DAsync(out_host->data, out_host->ld * oes, out_dev->data, out_dev->ld * oes, out_dev->cols * oes,
                                out_dev->rows, cudaMemcpyDeviceToHost, s));
  if (scale_len(*out_dev))
    HERO_CUDA(cudaMemcpyAsync(out_host->scale, out_dev->scale, scale_len(*out_dev) * sizeof(float), cudaMemcpyDeviceToHost, s));
  return HERO_OK;
}

// ---------------------------------------------------------------------------------------------------------------------
// A stack of layers: host-side sequencing of hero_layer_forward over chained edge tensors, with an optional entry LN^quant.
namespace hero {
static hero_status copy_tensor(const hero_tensor& dst, const hero_tensor& src, cudaMemcpyKind kind, cudaStream_t s, const char* what) {
  HERO_REQUIRE(dst.data && src.data && dst.dtype == src.dtype && dst.rows == src.rows && dst.cols == src.cols, HERO_ERR_INVALID_ARG,
               "%s: host and device tensors must agree in type and shape", what);
  const size_t es = dtype_size(dst.dtype);
  HERO_REQUIRE(es != 0, HERO_ERR_INVALID_ARG, "%s: unknown dtype", what);
  if (dst.ld == dst.cols && src.ld == src.cols)
    HERO_CUDA(cudaMemcpyAsync(dst.data, src.data, (size_t)dst.rows * dst.cols * es, kind, s));
  else
    HERO_CUDA(cudaMemcpy2DAsync(dst.data, dst.ld * es, src.data, src.ld * es, dst.cols * es, dst.rows, kind, s));
  if (is_q8(dst.dtype) && dst.gran == HERO_GRAN_TWQ) {      // token-wise scales travel with the payload; calibrated ones live on the device
    HERO_REQUIRE(dst.scale && src.scale, HERO_ERR_INVALID_ARG, "%s: a token-wise tensor needs its row scales on both sides", what);
    HERO_CUDA(cudaMemcpyAsync(dst.scale, src.scale, (size_t)dst.rows * sizeof(float), kind, s));
  }
  return HERO_OK;
}
}  // namespace hero

extern "C" hero_status hero_stack_forward(hero_handle* h, const hero_stack_desc* sd, void* workspace, size_t workspace_bytes,
                                          void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && sd && sd->n_layers > 0 && sd->layers && sd->edges, HERO_ERR_INVALID_ARG, "hero_stack_forward: bad stack descriptor");
  hero_status st;
  if (sd->entry_in.data) {
    hero_ln_args a;
    memset(&a, 0, sizeof(a));
    a.residual = sd->entry_in;
    a.gamma = sd->entry_gamma; a.beta = sd->entry_beta; a.eps = sd->entry_eps;
    a.out = sd->edges[0];
    if ((st = hero_layernorm_quant(h, &a, stream)) != HERO_OK) return st;
  }
  for (int32_t i = 0; i < sd->n_layers; ++i) {
    const hero_tensor* pend = (sd->pending && sd->pending[i].data) ? &sd->pending[i] : nullptr;
    if ((st = hero_layer_forward(h, &sd->layers[i], &sd->edges[i], pend, &sd->edges[i + 1], workspace, workspace_bytes, stream)) != HERO_OK)
      return st;
  }
  return HERO_OK;
}

extern "C" hero_status hero_stack_forward_host_async(hero_handle* h, const hero_stack_desc* sd, const hero_tensor* in_host,
                                                     const hero_tensor* out_host, void* workspace, size_t workspace_bytes,
                                                     void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && sd && in_host && out_host && sd->n_layers > 0 && sd->edges, HERO_ERR_INVALID_ARG,
               "hero_stack_forward_host: NULL argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  hero_status st;
  if ((st = copy_tensor(sd->entry_in.data ? sd->entry_in : sd->edges[0], *in_host, cudaMemcpyHostToDevice, s, "stack input")) != HERO_OK) return st;
  if ((st = hero_stack_forward(h, sd, workspace, workspace_bytes, stream)) != HERO_OK) return st;
  return copy_tensor(*out_host, sd->edges[sd->n_layers], cudaMemcpyDeviceToHost, s, "stack output");
}

extern "C" hero_status hero_layer_forward_host(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in_host,
                                               const hero_tensor* out_host, const hero_tensor* in_dev,
                                               const hero_tensor* out_dev, void* workspace, size_t workspace_bytes,
                                               void* stream) {
  hero_status st = hero_layer_forward_host_async(h, d, in_host, out_host, in_dev, out_dev, workspace, workspace_bytes, stream);
  if (st != HERO_OK) return st;
  HERO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return HERO_OK;
}
