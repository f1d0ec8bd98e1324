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
  int tma_out;              // the 8-bit output leaves through bulk tensor stores (CTA-pair kernel)
  float* obs_col;           // [N] or NULL: running per-column absmax of an FP output (calibration observer)
  int* err;
};

template <int BN>
struct GemmCfg {
  static constexpr int A_BYTES = GEMM_BM * GEMM_BK_BYTES;
  static constexpr int B_BYTES = BN * GEMM_BK_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int EPI_FLOATS = 4 * 3 * BN;                 // per-warp cs / bias / post
  static constexpr int SMEM_BYTES = 1024 /*align slack*/ + STAGES * STAGE_BYTES + EPI_FLOATS * 4 + 256 /*barriers*/;
};

constexpr float ROUND_MAGIC = 12582912.0f;   // 1.5 * 2^23

// GELU(v) = v Phi(v) = max(v, 0) - 0.5 a erfc(a / sqrt 2) with a = |v|.  log2 erfc(a / sqrt 2) is close to a parabola, so
// a degree-6 polynomial P(a) (fitted on [0, 6] with the weight a erfc: what an error in P does to the result) gives
// erfc(a / sqrt 2) = 2^P(a) with one special-function op per element and no reciprocal: absolute error of the GELU
// below 1.5e-7 everywhere (8.4e-8 from the polynomial in FP32 Horner form, the rest from ex2.approx).  Beyond a = 6 the
// term is below 1e-8 and a is clamped (the polynomial is not meant for larger arguments).  Branch-free, no
// cancellation for negative v.  Evaluated in n = -a (odd coefficients change sign) with the factor 0.5 folded into the
// constant term (P0 - 1), so that the result is one fused multiply-add: max(v, 0) + n 2^(P(a) - 1).
constexpr float GELU_P0 = 6.939127616e-06f, GELU_P1 = -1.151201725e+00f, GELU_P2 = -4.587709606e-01f,
                GELU_P3 = -5.341210961e-02f, GELU_P4 = 8.080720901e-03f, GELU_P5 = -7.692211657e-04f,
                GELU_P6 = 3.309298336e-05f;
__device__ __forceinline__ float gelu_erf_f(float v) {
  const float n = fmaxf(-fabsf(v), -6.0f);
  float q = fmaf(GELU_P6, n, -GELU_P5);
  q = fmaf(q, n, GELU_P4);
  q = fmaf(q, n, -GELU_P3);
  q = fmaf(q, n, GELU_P2);
  q = fmaf(q, n, -GELU_P1);
  q = fmaf(q, n, GELU_P0 - 1.0f);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(q));                   // 0.5 erfc(a / sqrt 2)
  return fmaf(n, e, fmaxf(v, 0.0f));
}
// the same on a packed pair: seven FFMA2, one special-function op per element
__device__ __forceinline__ float2 gelu_erf_f2(float2 v) {
  const float2 n = make_float2(fmaxf(-fabsf(v.x), -6.0f), fmaxf(-fabsf(v.y), -6.0f));
  float2 q = __ffma2_rn(make_float2(GELU_P6, GELU_P6), n, make_float2(-GELU_P5, -GELU_P5));
  q = __ffma2_rn(q, n, make_float2(GELU_P4, GELU_P4));
  q = __ffma2_rn(q, n, make_float2(-GELU_P3, -GELU_P3));
  q = __ffma2_rn(q, n, make_float2(GELU_P2, GELU_P2));
  q = __ffma2_rn(q, n, make_float2(-GELU_P1, -GELU_P1));
  q = __ffma2_rn(q, n, make_float2(GELU_P0 - 1.0f, GELU_P0 - 1.0f));
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(q.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(q.y));
  return __ffma2_rn(n, e, make_float2(fmaxf(v.x, 0.0f), fmaxf(v.y, 0.0f)));
}
__device__ __forceinline__ float gelu_tanh_f(float x) {
  return 0.5f * x * (1.0f + tanhf(0.79788456080286535588f * (x + 0.044715f * x * x * x)));
}

// few-row path (gemm_skinny.cu): M <= GEMM_BM, `p` filled by hero_w8a8_linear up to the tiling
hero_status run_skinny(hero_handle* h, const hero_linear_args* a, GemmParams& p, cudaStream_t s);

}  // namespace hero
