// Calibration on the GPU (Sec. 2.1, "calibration"; Eq. 2, Eq. 4-5, Eq. 20-23, Eq. 32): the statistics the static and
// feature-wise scales are made of, and the folding + column-wise quantization of the weights.
//
//   hero_absmax_observe  : running per-feature and per-tensor absmax of an FP16 / BF16 tensor at an operator border of
//                          the un-quantized (FP-mode) layer.  One streaming pass, 2 bytes per element: HBM-bound.
//   hero_quantize_weight : W~ = Diag(in_scale) W Diag(1 / out_scale), b~ = b / out_scale (fold first), then per output
//                          feature S_w = absmax / 127 and W_i8 = Round(W~ / S_w).  One CTA per output feature; the
//                          second sweep over the row hits L2.  4 bytes read + 1 written per weight: HBM-bound.
// The maximum softmax probability (S_p = max P / 255) is observed by the FP attention kernel itself.
#include "common.cuh"
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

// absmax values are non-negative floats: their bit patterns order like unsigned integers
__device__ __forceinline__ void atomic_max_nonneg(float* addr, float v) {
  // the running maximum only grows: a value that does not exceed what is already there needs no atomic
  if (v > __ldcg(addr)) atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

template <bool BF>
__device__ __forceinline__ void absmax8(const uint4 w, float (&m)[8]) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a, b;
    if constexpr (BF) { a = __uint_as_float(u[i] << 16); b = __uint_as_float(u[i] & 0xffff0000u); }
    else { const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&u[i])); a = f.x; b = f.y; }
    m[2 * i] = fmaxf(m[2 * i], fabsf(a));
    m[2 * i + 1] = fmaxf(m[2 * i + 1], fabsf(b));
  }
}

// blockDim = (CX, CY): CX threads cover 8 * CX consecutive columns (chunks of 8), CY rows at a time.  A thread walks
// the column chunks c = threadIdx.x, threadIdx.x + CX, ... and, for each, the rows of this CTA's strip, so that the
// running maxima stay in registers and every row segment is read with 16-byte loads, consecutive lanes adjacent.
template <bool BF>
__global__ void __launch_bounds__(256) absmax_kernel(const uint16_t* __restrict__ x, long long ld, long long rows, int cols,
                                                     long long rows_per_cta, float* col_absmax, float* tensor_absmax) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  const int nchunk = cols >> 3;
  const long long r0 = (long long)blockIdx.x * rows_per_cta;
  const long long r1 = min(rows, r0 + rows_per_cta);
  float tmax = 0.f;
  for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
    float m[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const uint16_t* col = x + (long long)c * 8;
    long long r = r0 + threadIdx.y;
    // four rows in flight per thread
    for (; r + 3 * (long long)blockDim.y < r1; r += 4 * (long long)blockDim.y) {
      uint4 w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = __ldg(reinterpret_cast<const uint4*>(col + (r + i * (long long)blockDim.y) * ld));
#pragma unroll
      for (int i = 0; i < 4; ++i) absmax8<BF>(w[i], m);
    }
    for (; r < r1; r += blockDim.y) absmax8<BF>(__ldg(reinterpret_cast<const uint4*>(col + r * ld)), m);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      tmax = fmaxf(tmax, m[i]);
      if (col_absmax && m[i] > 0.f) atomic_max_nonneg(col_absmax + c * 8 + i, m[i]);
    }
  }
  if (tensor_absmax) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    if (((threadIdx.y * blockDim.x + threadIdx.x) & 31) == 0 && tmax > 0.f) atomic_max_nonneg(tensor_absmax, tmax);
  }
}

// Histogram of |x| / bound over NBINS equal bins (values at or above the bound land in the last bin): per-CTA counts in
// shared memory, one global atomic per bin and CTA at the end.  The percentile clipping threshold of a static scale is
// read off the cumulative counts on the host.
constexpr int HIST_BINS = 2048;
template <bool BF>
__global__ void __launch_bounds__(256) abs_hist_kernel(const uint16_t* __restrict__ x, long long ld, long long rows, int cols,
                                                       long long rows_per_cta, float inv_bin, unsigned long long* hist) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  __shared__ unsigned int sh[HIST_BINS];
  for (int i = threadIdx.x; i < HIST_BINS; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const int nchunk = cols >> 3;
  const long long r0 = (long long)blockIdx.x * rows_per_cta, r1 = min(rows, r0 + rows_per_cta);
  for (long long r = r0; r < r1; ++r) {
    for (int c = threadIdx.x; c < nchunk; c += blockDim.x) {
      const uint4 w = __ldg(reinterpret_cast<const uint4*>(x + r * ld + (long long)c * 8));
      const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float a, b;
        if constexpr (BF) { a = __uint_as_float(u[i] << 16); b = __uint_as_float(u[i] & 0xffff0000u); }
        else { const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&u[i])); a = f.x; b = f.y; }
        atomicAdd(&sh[min(HIST_BINS - 1, (int)(fabsf(a) * inv_bin))], 1u);
        atomicAdd(&sh[min(HIST_BINS - 1, (int)(fabsf(b) * inv_bin))], 1u);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < HIST_BINS; i += blockDim.x)
    if (sh[i]) atomicAdd(hist + i, (unsigned long long)sh[i]);
}

// One CTA per output feature n: row n of W [N][K] (FP32).  F8: the e4m3 payload of the FP8 variant (scale absmax / 448,
// codes by the saturating round-to-nearest-even conversion) instead of INT8.
template <bool F8>
__global__ void __launch_bounds__(256) quantize_weight_kernel(const float* __restrict__ W, long long ldw, int N, int K,
                                                              const float* __restrict__ in_scale,
                                                              const float* __restrict__ out_scale,
                                                              const float* __restrict__ bias, int8_t* __restrict__ Wq,
                                                              long long ldq, float* __restrict__ w_scale,
                                                              float* __restrict__ bias_out) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  __shared__ float red[8];
  const int n = blockIdx.x;
  const float* row = W + (long long)n * ldw;
  const float o = out_scale ? out_scale[n] : 1.0f;              // the definition divides: kept as a division
  // ---- sweep 1: absmax of the folded row
  float m = 0.f;
  for (int k = threadIdx.x * 4; k < K; k += blockDim.x * 4) {
    const float4 w = __ldg(reinterpret_cast<const float4*>(row + k));
    float4 s = make_float4(1.f, 1.f, 1.f, 1.f);
    if (in_scale) s = __ldg(reinterpret_cast<const float4*>(in_scale + k));
    m = fmaxf(m, fmaxf(fmaxf(fabsf(w.x * s.x / o), fabsf(w.y * s.y / o)), fmaxf(fabsf(w.z * s.z / o), fabsf(w.w * s.w / o))));
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
  const float sw = m > 0.f ? m / (F8 ? 448.0f : 127.0f) : 1.0f;  // Eq. 2
  if (threadIdx.x == 0) {
    w_scale[n] = sw;
    if (bias_out) bias_out[n] = bias ? bias[n] / o : 0.f;
  }
  // ---- sweep 2: quantize (the row is in L2 now)
  int8_t* qrow = Wq + (long long)n * ldq;
  for (int k = threadIdx.x * 4; k < K; k += blockDim.x * 4) {
    const float4 w = __ldg(reinterpret_cast<const float4*>(row + k));
    float4 s = make_float4(1.f, 1.f, 1.f, 1.f);
    if (in_scale) s = __ldg(reinterpret_cast<const float4*>(in_scale + k));
    if constexpr (F8) {
      *reinterpret_cast<uint32_t*>(qrow + k) = ptx::f32x4_to_e4m3x4(w.x * s.x / o / sw, w.y * s.y / o / sw, w.z * s.z / o / sw, w.w * s.w / o / sw);
    } else {
      const int a = __float2int_rn(fminf(fmaxf(w.x * s.x / o / sw, -127.f), 127.f));
      const int b = __float2int_rn(fminf(fmaxf(w.y * s.y / o / sw, -127.f), 127.f));
      const int c = __float2int_rn(fminf(fmaxf(w.z * s.z / o / sw, -127.f), 127.f));
      const int d = __float2int_rn(fminf(fmaxf(w.w * s.w / o / sw, -127.f), 127.f));
      *reinterpret_cast<uint32_t*>(qrow + k) =
          (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) | ((uint32_t)d << 24);
    }
  }
}

}  // namespace hero

extern "C" hero_status hero_absmax_observe(hero_handle* h, const hero_tensor* x, float* col_absmax, float* tensor_absmax,
                                           void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && x, HERO_ERR_INVALID_ARG, "hero_absmax_observe: NULL handle or tensor");
  HERO_REQUIRE(col_absmax || tensor_absmax, HERO_ERR_INVALID_ARG, "neither col_absmax nor tensor_absmax given");
  hero_status st;
  if ((st = check_matrix(*x, "x")) != HERO_OK) return st;
  HERO_REQUIRE(is_fp16ish(x->dtype), HERO_ERR_UNSUPPORTED, "observers read F16 / BF16 tensors (the un-quantized layer)");
  HERO_REQUIRE(x->cols % 8 == 0 && x->ld % 8 == 0, HERO_ERR_ALIGNMENT, "cols and ld must be multiples of 8 elements");
  if (x->rows == 0) return HERO_OK;
  const int nchunk = (int)(x->cols / 8);
  int cx = 32;
  while (cx < 256 && cx < nchunk) cx *= 2;
  const int cy = 256 / cx;
  // strips of rows: about 8 CTAs per SM, at least 64 rows per thread row so that the final atomics stay rare
  long long ctas = (long long)h->sm_count * 8;
  long long rows_per_cta = (x->rows + ctas - 1) / ctas;
  const long long min_rows = 64LL * cy;
  if (rows_per_cta < min_rows) rows_per_cta = min_rows;
  ctas = (x->rows + rows_per_cta - 1) / rows_per_cta;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchScope scope(h, s, KERNEL_LN);
    if (x->dtype == HERO_BF16)
      HERO_CUDA(launch_dependent(absmax_kernel<true>, dim3((unsigned)ctas), dim3(cx, cy), 0, s,
                                 reinterpret_cast<const uint16_t*>(x->data), (long long)x->ld, (long long)x->rows,
                                 (int)x->cols, rows_per_cta, col_absmax, tensor_absmax));
    else
      HERO_CUDA(launch_dependent(absmax_kernel<false>, dim3((unsigned)ctas), dim3(cx, cy), 0, s,
                                 reinterpret_cast<const uint16_t*>(x->data), (long long)x->ld, (long long)x->rows,
                                 (int)x->cols, rows_per_cta, col_absmax, tensor_absmax));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

extern "C" hero_status hero_abs_histogram(hero_handle* h, const hero_tensor* x, float bound, uint64_t* hist, void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && x && hist, HERO_ERR_INVALID_ARG, "hero_abs_histogram: NULL argument");
  HERO_REQUIRE(bound > 0.f, HERO_ERR_INVALID_ARG, "bound must be positive");
  hero_status st;
  if ((st = check_matrix(*x, "x")) != HERO_OK) return st;
  HERO_REQUIRE(is_fp16ish(x->dtype), HERO_ERR_UNSUPPORTED, "observers read F16 / BF16 tensors (the un-quantized layer)");
  HERO_REQUIRE(x->cols % 8 == 0 && x->ld % 8 == 0, HERO_ERR_ALIGNMENT, "cols and ld must be multiples of 8 elements");
  if (x->rows == 0) return HERO_OK;
  long long ctas = (long long)h->sm_count * 8;
  long long rows_per_cta = (x->rows + ctas - 1) / ctas;
  if (rows_per_cta < 8) rows_per_cta = 8;
  ctas = (x->rows + rows_per_cta - 1) / rows_per_cta;
  const float inv_bin = (float)HIST_BINS / bound;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchScope scope(h, s, KERNEL_LN);
    if (x->dtype == HERO_BF16)
      HERO_CUDA(launch_dependent(abs_hist_kernel<true>, dim3((unsigned)ctas), dim3(256), 0, s,
                                 reinterpret_cast<const uint16_t*>(x->data), (long long)x->ld, (long long)x->rows, (int)x->cols,
                                 rows_per_cta, inv_bin, reinterpret_cast<unsigned long long*>(hist)));
    else
      HERO_CUDA(launch_dependent(abs_hist_kernel<false>, dim3((unsigned)ctas), dim3(256), 0, s,
                                 reinterpret_cast<const uint16_t*>(x->data), (long long)x->ld, (long long)x->rows, (int)x->cols,
                                 rows_per_cta, inv_bin, reinterpret_cast<unsigned long long*>(hist)));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

namespace hero {
static hero_status quantize_weight_impl(hero_handle* h, const float* W, int64_t ldw, int32_t N, int32_t K, const float* in_scale,
                                        const float* out_scale, const float* bias, void* Wq, int64_t ldq, float* w_scale,
                                        float* bias_out, bool f8, void* stream) {
  HERO_REQUIRE(h && W && Wq && w_scale, HERO_ERR_INVALID_ARG, "hero_quantize_weight: NULL argument");
  HERO_REQUIRE(N >= 0 && K > 0 && K % 4 == 0 && ldw >= K && ldw % 4 == 0 && ldq >= K && ldq % 4 == 0, HERO_ERR_INVALID_ARG,
               "K, ldw and ldq must be positive multiples of 4 with ld >= K");
  HERO_REQUIRE(aligned16(W) && (!in_scale || aligned16(in_scale)) && (reinterpret_cast<uintptr_t>(Wq) & 3) == 0,
               HERO_ERR_ALIGNMENT, "W and in_scale must be 16-byte aligned, Wq 4-byte aligned");
  if (N == 0) return HERO_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    LaunchScope scope(h, s, KERNEL_GEMM);
    auto kern = f8 ? quantize_weight_kernel<true> : quantize_weight_kernel<false>;
    HERO_CUDA(launch_dependent(kern, dim3((unsigned)N), dim3(256), 0, s, W, (long long)ldw, (int)N, (int)K, in_scale, out_scale,
                               bias, static_cast<int8_t*>(Wq), (long long)ldq, w_scale, bias_out));
  }
  pdl_fence_stream(s);   // Wq, w_scale and bias_out are model constants to whatever runs next on this stream
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}
}  // namespace hero

extern "C" hero_status hero_quantize_weight(hero_handle* h, const float* W, int64_t ldw, int32_t N, int32_t K,
                                            const float* in_scale, const float* out_scale, const float* bias,
                                            int8_t* Wq, int64_t ldq, float* w_scale, float* bias_out, void* stream) {
  return hero::quantize_weight_impl(h, W, ldw, N, K, in_scale, out_scale, bias, Wq, ldq, w_scale, bias_out, false, stream);
}

extern "C" hero_status hero_quantize_weight_f8(hero_handle* h, const float* W, int64_t ldw, int32_t N, int32_t K,
                                               const float* in_scale, const float* out_scale, const float* bias,
                                               uint8_t* Wq, int64_t ldq, float* w_scale, float* bias_out, void* stream) {
  return hero::quantize_weight_impl(h, W, ldw, N, K, in_scale, out_scale, bias, Wq, ldq, w_scale, bias_out, true, stream);
}
