// Shared by the GeMM^quant kernels (Sec. 2.2.2 Eq. 14, 18, 20-23; Sec. 2.2.3 Eq. 28-30, 32): launch parameters, tile
// constants and the activation functions of the fused epilogue.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK_BYTES = 128;   // one swizzle row
constexpr int GEMM_THREADS = 320;
constexpr int TMA_WARP = 8, MMA_WARP = 9;
constexpr int OUT_I8 = 0, OUT_FP = 1, OUT_I32 = 2, OUT_F8 = 3;

struct GemmParams {
  int M, N, K;              // K in elements
  int num_m_tiles, num_n_tiles, num_kb;
  const float* rs;          // [M] or NULL
  const float* cs;          // [N] or NULL (FP operands)
  const float* bias;        // [N] or NULL
  const float* post;        // [N] or NULL
  void* out;
  long long out_ld;         // elements
  int out_dt;               // hero_dtype
  uint32_t idesc;
  int elem_bytes;           // 1 (INT8, e4m3) or 2 (F16 / BF16)
  int f8;                   // operands are e4m3 (kind::f8f6f4; FP32 accumulators, scales as for INT8)
  int* err;
};

template <int BN>
struct GemmCfg {
  static constexpr int A_BYTES = GEMM_BM * GEMM_BK_BYTES;
  static constexpr int B_BYTES = BN * GEMM_BK_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int EPI_FLOATS = 4 * 2 * 3 * BN;             // per-warp, double-buffered cs / bias / post
  static constexpr int SMEM_BYTES = 1024 /*align slack*/ + STAGES * STAGE_BYTES + EPI_FLOATS * 4 + 256 /*barriers*/;
};

constexpr float ROUND_MAGIC = 12582912.0f;   // 1.5 * 2^23

// GELU(v) = v Phi(v) = max(v, 0) - 0.5 |v| E(|v| / sqrt 2) with E(z) = erfc(z) for z >= 0, evaluated with the
// rational-exponential form erfc(z) ~ (a1 t + ... + a5 t^5) exp(-z^2), t = 1 / (1 + p z) (absolute error
// below 1.5e-7 for every z >= 0): branch-free, two special-function ops, no cancellation for negative v.
__device__ __forceinline__ float gelu_erf_f(float v) {
  const float av = fabsf(v);
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(av, 0.3275911f * 0.70710678118654752440f, 1.0f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  poly *= t;
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(v * v * -0.72134752044448170368f));   // exp(-v^2 / 2)
  return fmaf(-0.5f * av, poly * e, fmaxf(v, 0.0f));
}
// the same on a packed pair: the polynomial and the products run as FFMA2 / FMUL2, two special-function ops per element
__device__ __forceinline__ float2 gelu_erf_f2(float2 v) {
  const float2 av = make_float2(fabsf(v.x), fabsf(v.y));
  const float kz = 0.3275911f * 0.70710678118654752440f;
  const float2 d = __ffma2_rn(av, make_float2(kz, kz), make_float2(1.0f, 1.0f));
  float2 t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.x) : "f"(d.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.y) : "f"(d.y));
  float2 poly = __ffma2_rn(make_float2(1.061405429f, 1.061405429f), t, make_float2(-1.453152027f, -1.453152027f));
  poly = __ffma2_rn(poly, t, make_float2(1.421413741f, 1.421413741f));
  poly = __ffma2_rn(poly, t, make_float2(-0.284496736f, -0.284496736f));
  poly = __ffma2_rn(poly, t, make_float2(0.254829592f, 0.254829592f));
  poly = __fmul2_rn(poly, t);
  const float2 q = __fmul2_rn(__fmul2_rn(v, make_float2(-0.72134752044448170368f, -0.72134752044448170368f)), v);
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(q.x));                // exp(-v^2 / 2)
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(q.y));
  const float2 w = __fmul2_rn(__fmul2_rn(av, make_float2(-0.5f, -0.5f)), __fmul2_rn(poly, e));
  return __fadd2_rn(w, make_float2(fmaxf(v.x, 0.0f), fmaxf(v.y, 0.0f)));
}
__device__ __forceinline__ float gelu_tanh_f(float x) {
  return 0.5f * x * (1.0f + tanhf(0.79788456080286535588f * (x + 0.044715f * x * x * x)));
}

// few-row path (gemm_skinny.cu): M <= GEMM_BM, `p` filled by hero_w8a8_linear up to the tiling
hero_status run_skinny(hero_handle* h, const hero_linear_args* a, GemmParams& p, cudaStream_t s);

}  // namespace hero
