// LN^quant family (Sec. 2.2.1 Eq. 6-7, Sec. 2.2.2 Eq. 19, Sec. 2.2.3 Eq. 31): one pass over each row.
//
// HBM-bound streaming kernel.  A row of H elements is owned by G = ceil(H / VEC) threads (rounded up
// to whole warps), each holding VEC consecutive elements in registers; a CTA of about 256 threads
// works on RPC = 256 / G rows at once and every thread keeps R rows in flight per loop trip so that
// enough 16-byte loads are outstanding to cover DRAM latency.  Row statistics are two-pass over the
// registers (mean, then centred variance), reduced with warp shuffles and, when a row spans several
// warps, one shared-memory exchange per statistic.  gamma / beta stay in registers across the
// persistent row loop; per-feature scale vectors are re-read through L1.
#include "common.cuh"
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

struct LnSide {           // one addend of the LayerNorm input
  const void* data;       // NULL = absent
  int dt;                 // hero_dtype
  long long ld;           // elements
  const float* row_scale; // TWQ scale [rows] or NULL
  const float* col_scale; // FWQ [H] (stride 1) or SQ [1] (stride 0) or NULL
  int col_stride;
};

struct LnParams {
  LnSide res, br, ex;
  const int* token_ids;   // embedding gather (Eq. 7) when non-NULL
  const int* type_ids;
  int seq_len;
  int n_tok_rows, n_type_rows;   // rows of the token / sentence-type tables: ids are clamped into them
  int* err;                      // device error word: an out-of-range id records ERR_BAD_ID there
  const float* gamma;
  const float* beta;
  float eps;
  void* out; int out_dt; long long out_ld; int out_gran; float* out_scale;
  void* fp_out; int fp_dt; long long fp_ld;
  float* obs;             // calibration: per-column running absmax of the FP tensor the call stores, or NULL
  long long M; int H;
  int G;                  // threads per row (multiple of 32)
  int RPC;                // rows per CTA per pass
};

// Row of an embedding table named by ids[row].  An id outside [0, n_rows) must not become an out-of-bounds read:
// it is clamped into the table and a code is left in the device error word for hero_check to report.
__device__ __forceinline__ long long table_row(const int* ids, long long row, int n_rows, int* err) {
  int id = ids[row];
  if ((unsigned)id >= (unsigned)n_rows) {
    if (err) atomicExch(err, ERR_BAD_ID);
    id = id < 0 ? 0 : n_rows - 1;
  }
  return id;
}

template <int VEC>
__device__ __forceinline__ void load_raw(const void* p, int bytes_per_elem, uint32_t (&w)[VEC / 2]) {
  // VEC elements of 1 or 2 bytes -> VEC/4 or VEC/2 32-bit words, streamed past L1
  if (bytes_per_elem == 1) {
    if constexpr (VEC == 8) {
      asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(p));
    } else {
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p));
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC / 8; ++i)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(w[4 * i]), "=r"(w[4 * i + 1]), "=r"(w[4 * i + 2]), "=r"(w[4 * i + 3])
                   : "l"(reinterpret_cast<const char*>(p) + 16 * i));
  }
}

template <int VEC>
__device__ __forceinline__ void unpack(const uint32_t (&w)[VEC / 2], int dt, float (&v)[VEC]) {
  if (dt == HERO_I8) {
#pragma unroll
    for (int i = 0; i < VEC / 4; ++i) {
#pragma unroll
      for (int b = 0; b < 4; ++b) v[4 * i + b] = (float)(int)(signed char)((w[i] >> (8 * b)) & 0xff);
    }
  } else if (dt == HERO_F8) {
#pragma unroll
    for (int i = 0; i < VEC / 4; ++i) {
      const float2 lo = ptx::e4m3x2_to_f32x2(w[i] & 0xffffu), hi = ptx::e4m3x2_to_f32x2(w[i] >> 16);
      v[4 * i] = lo.x; v[4 * i + 1] = lo.y; v[4 * i + 2] = hi.x; v[4 * i + 3] = hi.y;
    }
  } else if (dt == HERO_F16) {
#pragma unroll
    for (int i = 0; i < VEC / 2; ++i) {
      float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC / 2; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
}

__device__ __forceinline__ uint32_t pack_fp2(float a, float b, int dt) {
  if (dt == HERO_F16) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d) {
  // clip(Round(.)) to [-127, 127], round-half-to-even, packed little-endian
  int ia = __float2int_rn(fminf(fmaxf(a, -127.f), 127.f));
  int ib = __float2int_rn(fminf(fmaxf(b, -127.f), 127.f));
  int ic = __float2int_rn(fminf(fmaxf(c, -127.f), 127.f));
  int id = __float2int_rn(fminf(fmaxf(d, -127.f), 127.f));
  return (uint32_t)(ia & 0xff) | ((uint32_t)(ib & 0xff) << 8) | ((uint32_t)(ic & 0xff) << 16) | ((uint32_t)id << 24);
}

template <int VEC>
__device__ __forceinline__ void store_words(void* p, const uint32_t* w, int nwords) {
  // nwords in {2, 4, 8}
  if (nwords == 2) {
    asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(w[0]), "r"(w[1]) : "memory");
  } else {
#pragma unroll
    for (int i = 0; i < nwords / 4; ++i)
      asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(reinterpret_cast<char*>(p) + 16 * i), "r"(w[4 * i]),
                   "r"(w[4 * i + 1]), "r"(w[4 * i + 2]), "r"(w[4 * i + 3])
                   : "memory");
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Reduce R per-thread values over the G threads of a row.  red: [RPC][R][G/32] floats.
template <int R, bool IS_MAX>
__device__ __forceinline__ void row_reduce(float (&v)[R], float* red, int G, int row_in_cta, int t) {
#pragma unroll
  for (int r = 0; r < R; ++r) v[r] = IS_MAX ? warp_max(v[r]) : warp_sum(v[r]);
  const int nw = G >> 5;
  if (nw == 1) return;
  float* mine = red + (size_t)row_in_cta * R * nw;
  if ((t & 31) == 0) {
#pragma unroll
    for (int r = 0; r < R; ++r) mine[r * nw + (t >> 5)] = v[r];
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float a = mine[r * nw];
    for (int w = 1; w < nw; ++w) a = IS_MAX ? fmaxf(a, mine[r * nw + w]) : a + mine[r * nw + w];
    v[r] = a;
  }
}

template <int VEC, int R, bool HAS_BR, bool HAS_EX>
__global__ void __launch_bounds__(1024) ln_quant_kernel(const LnParams p) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();                                 // the previous kernel's outputs are complete and visible
  extern __shared__ float red_smem[];
  const int G = p.G, RPC = p.RPC, H = p.H;
  const int nw = G >> 5;
  float* red0 = red_smem;
  float* red1 = red0 + RPC * R * nw;
  float* red2 = red1 + RPC * R * nw;

  const int tid = threadIdx.x;
  const int row_in_cta = tid / G;
  const int t = tid - row_in_cta * G;
  const int c0 = t * VEC;
  const bool active = c0 < H;

  float gam[VEC], bet[VEC];
  const bool normalize = p.out != nullptr;
  if (active && normalize) {
#pragma unroll
    for (int i = 0; i < VEC; i += 4) {
      float4 g4 = *reinterpret_cast<const float4*>(p.gamma + c0 + i);
      float4 b4 = *reinterpret_cast<const float4*>(p.beta + c0 + i);
      gam[i] = g4.x; gam[i + 1] = g4.y; gam[i + 2] = g4.z; gam[i + 3] = g4.w;
      bet[i] = b4.x; bet[i + 1] = b4.y; bet[i + 2] = b4.z; bet[i + 3] = b4.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC; ++i) { gam[i] = 0.f; bet[i] = 0.f; }
  }

  const int res_es = is_q8(p.res.dt) ? 1 : 2;
  const int br_es = is_q8(p.br.dt) ? 1 : 2;
  const long long rows_per_trip = (long long)RPC * R;
  float om[VEC];          // calibration observer: this thread's columns, maximum over the rows it visits
#pragma unroll
  for (int i = 0; i < VEC; ++i) om[i] = 0.f;

  for (long long base = (long long)blockIdx.x * rows_per_trip; base < p.M; base += (long long)gridDim.x * rows_per_trip) {
    float x[R][VEC];
    uint32_t raw_res[R][VEC / 2], raw_br[HAS_BR ? R : 1][VEC / 2], raw_ex[HAS_EX ? R : 1][VEC / 2];
    long long row[R];
    bool valid[R];
    float rs_res[R], rs_br[R];

    // ---- issue every load of the trip before touching the data
#pragma unroll
    for (int r = 0; r < R; ++r) {
      row[r] = base + (long long)r * RPC + row_in_cta;
      valid[r] = active && row[r] < p.M;
      rs_res[r] = 1.f; rs_br[r] = 1.f;
      if (valid[r]) {
        long long rr = row[r], rb = row[r], re = row[r];
        if (p.token_ids) {
          rr = table_row(p.token_ids, row[r], p.n_tok_rows, p.err);
          rb = row[r] % p.seq_len;
          re = p.type_ids ? table_row(p.type_ids, row[r], p.n_type_rows, p.err) : 0;
        }
        load_raw<VEC>(reinterpret_cast<const char*>(p.res.data) + (rr * p.res.ld + c0) * res_es, res_es, raw_res[r]);
        if (p.res.row_scale) rs_res[r] = p.res.row_scale[rr];
        if constexpr (HAS_BR) {
          load_raw<VEC>(reinterpret_cast<const char*>(p.br.data) + (rb * p.br.ld + c0) * br_es, br_es, raw_br[r]);
          if (p.br.row_scale) rs_br[r] = p.br.row_scale[rb];
        }
        if constexpr (HAS_EX)
          load_raw<VEC>(reinterpret_cast<const char*>(p.ex.data) + (re * p.ex.ld + c0) * 2, 2, raw_ex[r]);
      }
    }

    // ---- r = sum of the dequantized addends (fp32)
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (valid[r]) {
        unpack<VEC>(raw_res[r], p.res.dt, x[r]);
        if (is_q8(p.res.dt)) {
          if (p.res.col_scale) {
#pragma unroll
            for (int i = 0; i < VEC; ++i) x[r][i] *= rs_res[r] * __ldg(p.res.col_scale + (c0 + i) * p.res.col_stride);
          } else {
#pragma unroll
            for (int i = 0; i < VEC; ++i) x[r][i] *= rs_res[r];
          }
        }
        if constexpr (HAS_BR) {
          float b[VEC];
          unpack<VEC>(raw_br[r], p.br.dt, b);
          if (is_q8(p.br.dt)) {
            if (p.br.col_scale) {
#pragma unroll
              for (int i = 0; i < VEC; ++i)
                x[r][i] = fmaf(b[i], rs_br[r] * __ldg(p.br.col_scale + (c0 + i) * p.br.col_stride), x[r][i]);
            } else {
#pragma unroll
              for (int i = 0; i < VEC; ++i) x[r][i] = fmaf(b[i], rs_br[r], x[r][i]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < VEC; ++i) x[r][i] += b[i];
          }
        }
        if constexpr (HAS_EX) {
          float e[VEC];
          unpack<VEC>(raw_ex[r], p.ex.dt, e);
#pragma unroll
          for (int i = 0; i < VEC; ++i) x[r][i] += e[i];
        }
        if (p.fp_out) {
          // the FP residual stream carries the ROUNDED sum; normalise what is stored
          uint32_t w[VEC / 2];
#pragma unroll
          for (int i = 0; i < VEC / 2; ++i) w[i] = pack_fp2(x[r][2 * i], x[r][2 * i + 1], p.fp_dt);
          store_words<VEC>(reinterpret_cast<char*>(p.fp_out) + (row[r] * p.fp_ld + c0) * 2, w, VEC / 2);
          unpack<VEC>(w, p.fp_dt, x[r]);
          if (p.obs && !normalize) {
#pragma unroll
            for (int i = 0; i < VEC; ++i) om[i] = fmaxf(om[i], fabsf(x[r][i]));
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) x[r][i] = 0.f;
      }
    }
    if (!normalize) continue;

    // ---- mean, then centred (biased) variance, both over registers
    float s[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float a = 0.f;
#pragma unroll
      for (int i = 0; i < VEC; ++i) a += x[r][i];
      s[r] = a;
    }
    row_reduce<R, false>(s, red0, G, row_in_cta, t);
    float mean[R], rstd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      mean[r] = s[r] / (float)H;
      float a = 0.f;
      if (active) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) { float d = x[r][i] - mean[r]; a = fmaf(d, d, a); }
      }
      s[r] = a;
    }
    row_reduce<R, false>(s, red1, G, row_in_cta, t);
#pragma unroll
    for (int r = 0; r < R; ++r) rstd[r] = 1.0f / sqrtf(s[r] / (float)H + p.eps);

    // ---- y = (x - mean) * rstd * gamma + beta
    float amax[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float m = 0.f;
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        float y = fmaf((x[r][i] - mean[r]) * rstd[r], gam[i], bet[i]);
        x[r][i] = y;
        m = fmaxf(m, fabsf(y));
      }
      amax[r] = m;
    }

    if (is_q8(p.out_dt)) {
      const bool f8 = p.out_dt == HERO_F8;
      float inv[R];
      if (p.out_gran == HERO_GRAN_TWQ) {
        // Eq. 3: S[i] = absmax / 127 (absmax / 448 for an e4m3 payload) computed on the fly, in the same pass
        row_reduce<R, true>(amax, red2, G, row_in_cta, t);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float sc = amax[r] > 0.f ? amax[r] / (f8 ? 448.0f : 127.0f) : 1.0f;
          inv[r] = 1.0f / sc;
          if (t == 0 && row[r] < p.M) p.out_scale[row[r]] = sc;
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!valid[r]) continue;
        uint32_t w[VEC / 4];
        if (p.out_gran == HERO_GRAN_TWQ) {
#pragma unroll
          for (int i = 0; i < VEC / 4; ++i) {
            const float a = x[r][4 * i] * inv[r], b = x[r][4 * i + 1] * inv[r], c = x[r][4 * i + 2] * inv[r], d = x[r][4 * i + 3] * inv[r];
            w[i] = f8 ? ptx::f32x4_to_e4m3x4(a, b, c, d) : quant4(a, b, c, d);
          }
        } else {
          // Eq. 4 / 5: calibrated per-feature (stride 1) or static (stride 0) scale
          const int st = (p.out_gran == HERO_GRAN_FWQ) ? 1 : 0;
          float q[VEC];
#pragma unroll
          for (int i = 0; i < VEC; ++i) q[i] = x[r][i] / __ldg(p.out_scale + (c0 + i) * st);
#pragma unroll
          for (int i = 0; i < VEC / 4; ++i)
            w[i] = f8 ? ptx::f32x4_to_e4m3x4(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3])
                      : quant4(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
        }
        store_words<VEC>(reinterpret_cast<char*>(p.out) + row[r] * p.out_ld + c0, w, VEC / 4);
      }
    } else {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!valid[r]) continue;
        uint32_t w[VEC / 2];
#pragma unroll
        for (int i = 0; i < VEC / 2; ++i) w[i] = pack_fp2(x[r][2 * i], x[r][2 * i + 1], p.out_dt);
        store_words<VEC>(reinterpret_cast<char*>(p.out) + (row[r] * p.out_ld + c0) * 2, w, VEC / 2);
        if (p.obs) {        // what is observed is what is stored: the rounded values
          float y[VEC];
          unpack<VEC>(w, p.out_dt, y);
#pragma unroll
          for (int i = 0; i < VEC; ++i) om[i] = fmaxf(om[i], fabsf(y[i]));
        }
      }
    }
  }
  if (p.obs && active) {    // non-negative floats order like their bit patterns
#pragma unroll
    for (int i = 0; i < VEC; ++i)
      if (om[i] > 0.f) atomicMax(reinterpret_cast<int*>(p.obs) + c0 + i, __float_as_int(om[i]));
  }
}

static hero_status fill_side(const hero_tensor& t, LnSide* s, const char* name, bool allow_i8, int H) {
  s->data = nullptr; s->dt = HERO_F16; s->ld = 0; s->row_scale = nullptr; s->col_scale = nullptr; s->col_stride = 0;
  if (t.data == nullptr) return HERO_OK;
  hero_status st = check_matrix(t, name);
  if (st != HERO_OK) return st;
  HERO_REQUIRE(t.cols == H, HERO_ERR_INVALID_ARG, "%s: cols %lld != H %d", name, (long long)t.cols, H);
  HERO_REQUIRE(is_fp16ish(t.dtype) || (allow_i8 && is_q8(t.dtype)), HERO_ERR_UNSUPPORTED,
               "%s: dtype %d not accepted here", name, t.dtype);
  s->data = t.data; s->dt = t.dtype; s->ld = t.ld;
  if (is_q8(t.dtype)) {
    if (t.gran == HERO_GRAN_TWQ) s->row_scale = t.scale;
    if (t.gran == HERO_GRAN_FWQ) { s->col_scale = t.scale; s->col_stride = 1; }
    if (t.gran == HERO_GRAN_SQ) { s->col_scale = t.scale; s->col_stride = 0; }
  }
  return HERO_OK;
}

template <int VEC, int R, bool HAS_BR, bool HAS_EX>
static hero_status launch_ln2(hero_handle* h, LnParams& p, cudaStream_t stream) {
  const int chunks = (p.H + VEC - 1) / VEC;
  p.G = ((chunks + 31) / 32) * 32;
  p.RPC = p.G >= 256 ? 1 : 256 / p.G;
  const int threads = p.G * p.RPC;
  const size_t smem = (size_t)3 * p.RPC * R * (p.G / 32) * sizeof(float);
  const long long rows_per_trip = (long long)p.RPC * R;
  long long want = (p.M + rows_per_trip - 1) / rows_per_trip;
  // a few CTAs per SM, persistent over the rows
  int occ = 1;
  HERO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, ln_quant_kernel<VEC, R, HAS_BR, HAS_EX>, threads, smem));
  if (occ < 1) occ = 1;
  long long cap = (long long)h->sm_count * occ;
  int grid = (int)(want < cap ? want : cap);
  if (grid < 1) grid = 1;
  {
    LaunchScope scope(h, stream, KERNEL_LN);
    HERO_CUDA(launch_dependent(ln_quant_kernel<VEC, R, HAS_BR, HAS_EX>, dim3(grid), dim3(threads), smem, stream, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

template <int VEC, int R>
static hero_status launch_ln(hero_handle* h, LnParams& p, cudaStream_t stream) {
  if (p.ex.data) return launch_ln2<VEC, R, true, true>(h, p, stream);   // embedding flavour: three addends
  if (p.br.data) return launch_ln2<VEC, R, true, false>(h, p, stream);  // residual flavour: two addends
  return launch_ln2<VEC, R, false, false>(h, p, stream);                // plain flavour
}


__device__ __forceinline__ void st_global8(void* p, uint32_t a, uint32_t b) {
  asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void st_global16(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// =====================================================================================================
// Fast path: types fixed at compile time, a row owned by WPR whole warps (H <= 1024 * WPR), each lane
// holding up to four 8-element chunks.  INT8 payloads are turned into floats with byte permutes and an
// exact float subtraction (no I2F), and the TWQ output is rounded with the 1.5 * 2^23 magic constant
// inside one FMA (no F2I): both keep the per-element instruction count low enough for the kernel to
// stay memory-bound.  gamma / beta / per-feature scales come through L1.
// =====================================================================================================
constexpr int SRC_NONE = 0, SRC_I8 = 1, SRC_FP = 2;
constexpr int O_NONE = 0, O_TWQ = 1, O_STATIC = 2, O_FP = 3;
constexpr int LNF_THREADS = 256;
constexpr int LNF_MAXCH = 4;

__device__ __forceinline__ void ldg8(const void* p, uint32_t& a, uint32_t& b) {
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(a), "=r"(b) : "l"(p));
}
__device__ __forceinline__ void ldg16(const void* p, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "l"(p));
}
__device__ __forceinline__ float4 ldg_f4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// 8 INT8 codes (two words) -> 8 exact floats
__device__ __forceinline__ void i8x8_to_float(uint32_t w0, uint32_t w1, float (&v)[8]) {
  w0 ^= 0x80808080u; w1 ^= 0x80808080u;           // code + 128 in [1, 255]
  const float off = 8388736.0f;                   // 2^23 + 128
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    v[b] = __uint_as_float(__byte_perm(w0, 0x4B000000u, 0x7440 | b)) - off;
    v[4 + b] = __uint_as_float(__byte_perm(w1, 0x4B000000u, 0x7440 | b)) - off;
  }
}
__device__ __forceinline__ void fp16x8_to_float(const uint32_t (&w)[4], int dt, float (&v)[8]) {
  if (dt == HERO_F16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
}
// Round-half-to-even of |v| <= 127.x through the float adder, low byte = two's complement code
__device__ __forceinline__ uint32_t magic_bits(float v_plus_magic) { return __float_as_uint(v_plus_magic); }
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  uint32_t ab = __byte_perm(a, b, 0x0040);        // bytes: a0, b0
  uint32_t cd = __byte_perm(c, d, 0x0040);
  return __byte_perm(ab, cd, 0x5410);
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int LNF_MAX_STAGES = 8; // ring depth is chosen at launch so that ~128 KB per SM are in flight

// Packed FP32 pairs: sm_100 issues add / mul / fma on two floats per instruction, which halves the issue
// slots of the arithmetic below (the kernel is bound by instruction issue, not by any one pipe).
__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }
__device__ __forceinline__ void load_vec8(const float* p, float2 (&v)[4]) {
  const float4 a = ldg_f4(p), b = ldg_f4(p + 4);
  v[0] = make_float2(a.x, a.y); v[1] = make_float2(a.z, a.w); v[2] = make_float2(b.x, b.y); v[3] = make_float2(b.z, b.w);
}
// 8 INT8 codes -> 4 float pairs (exact): byte + 128 into the mantissa of 2^23, then one packed subtraction
__device__ __forceinline__ void i8x8_to_f2(uint32_t w0, uint32_t w1, float2 (&v)[4]) {
  w0 ^= 0x80808080u; w1 ^= 0x80808080u;
  const float2 off = f2(-8388736.0f);             // -(2^23 + 128)
  v[0] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(w0, 0x4B000000u, 0x7440)), __uint_as_float(__byte_perm(w0, 0x4B000000u, 0x7441))), off);
  v[1] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(w0, 0x4B000000u, 0x7442)), __uint_as_float(__byte_perm(w0, 0x4B000000u, 0x7443))), off);
  v[2] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(w1, 0x4B000000u, 0x7440)), __uint_as_float(__byte_perm(w1, 0x4B000000u, 0x7441))), off);
  v[3] = __fadd2_rn(make_float2(__uint_as_float(__byte_perm(w1, 0x4B000000u, 0x7442)), __uint_as_float(__byte_perm(w1, 0x4B000000u, 0x7443))), off);
}
__device__ __forceinline__ void fp16x8_to_f2(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, int dt, float2 (&v)[4]) {
  const uint32_t w[4] = {w0, w1, w2, w3};
  if (dt == HERO_F16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
  }
}

// NCHX = exact number of 8-element chunks per lane (H = 256 * WPR * NCHX, no tail predicates), or 0 for any H.
template <int RES, int BR, bool EX, int OUT, bool FPOUT, int NCHX>
__global__ void __launch_bounds__(LNF_THREADS, 2) ln_fast_kernel(const LnParams p) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();                                 // the previous kernel's outputs are complete and visible
  constexpr int KMAX = NCHX ? NCHX : LNF_MAXCH;
  // gamma / beta (and, with at most 3 chunks per lane, the branch's per-feature scale) stay in registers for
  // the whole persistent row loop of the exact-size variants; otherwise they are re-read through L1 per row
  constexpr bool GB_REG = NCHX != 0;
  constexpr bool CS_REG = (NCHX == 2 || NCHX == 3) && BR == SRC_I8;
  auto chunk_ok = [&](int c) -> bool { if constexpr (NCHX != 0) return true; else return c < (p.H >> 3); };
  __shared__ float red[3][8][8];                  // [statistic][row slot][warp in row]
  extern __shared__ __align__(16) uint8_t ring[]; // [stage][row slot][res row | branch row | extra row]
  const int WPR = p.G;                            // warps per row: 1, 2, 4 or 8
  const int slots = 8 / WPR;                      // rows per CTA pass
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slot = warp / WPR, wr = warp - slot * WPR;
  const int stride = WPR * 32;                    // chunk stride between a lane's chunks
  const int c_first = wr * 32 + lane;
  const float fH = (float)p.H;
  const float MAGIC = 12582912.0f;                // 1.5 * 2^23
  constexpr int ES_RES = (RES == SRC_I8) ? 1 : 2;
  constexpr int ES_BR = (BR == SRC_I8) ? 1 : (BR == SRC_FP ? 2 : 0);
  const int off_br = p.H * ES_RES;
  const int off_ex = off_br + p.H * ES_BR;
  const int slot_bytes = off_ex + (EX ? p.H * 2 : 0);
  const int stage_bytes = slot_bytes * slots;
  const int STAGES = p.RPC;                       // ring depth (3..8), chosen by the host

  // A lane copies exactly the chunks it will later read, so waiting on its own copy groups is all
  // the synchronisation the ring needs.
  auto prefetch = [&](long long row, int st) {
    if (row < p.M) {
      long long r_res = row, r_br = row, r_ex = row;
      if constexpr (EX) {
        if (p.token_ids) {
          r_res = table_row(p.token_ids, row, p.n_tok_rows, p.err);
          r_br = row % p.seq_len;
          r_ex = p.type_ids ? table_row(p.type_ids, row, p.n_type_rows, p.err) : 0;
        }
      }
      uint8_t* dst = ring + st * stage_bytes + slot * slot_bytes;
      const char* g_res = reinterpret_cast<const char*>(p.res.data) + r_res * p.res.ld * ES_RES;
      const char* g_br = (BR != SRC_NONE) ? reinterpret_cast<const char*>(p.br.data) + r_br * p.br.ld * ES_BR : nullptr;
      const char* g_ex = EX ? reinterpret_cast<const char*>(p.ex.data) + r_ex * p.ex.ld * 2 : nullptr;
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        const int c = c_first + k * stride;
        if (chunk_ok(c)) {
          if constexpr (RES == SRC_I8) cp_async8(dst + c * 8, g_res + c * 8);
          else cp_async16(dst + c * 16, g_res + c * 16);
          if constexpr (BR == SRC_I8) cp_async8(dst + off_br + c * 8, g_br + c * 8);
          if constexpr (BR == SRC_FP) cp_async16(dst + off_br + c * 16, g_br + c * 16);
          if constexpr (EX) cp_async16(dst + off_ex + c * 16, g_ex + c * 16);
        }
      }
    }
    cp_async_commit();
  };

  const long long row_step = (long long)gridDim.x * slots;
  const long long first = (long long)blockIdx.x * slots;
  for (int s0 = 0; s0 < STAGES - 1; ++s0) prefetch(first + s0 * row_step + slot, s0);

  float2 gam[GB_REG ? KMAX : 1][4], bet[GB_REG ? KMAX : 1][4], bcs[CS_REG ? KMAX : 1][4];
  if constexpr (GB_REG && OUT != O_NONE) {
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      load_vec8(p.gamma + (c_first + k * stride) * 8, gam[k]);
      load_vec8(p.beta + (c_first + k * stride) * 8, bet[k]);
    }
  }
  if constexpr (CS_REG) {
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int c8 = (c_first + k * stride) * 8;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        bcs[k][i].x = p.br.col_scale ? __ldg(p.br.col_scale + (c8 + 2 * i) * p.br.col_stride) : 1.0f;
        bcs[k][i].y = p.br.col_scale ? __ldg(p.br.col_scale + (c8 + 2 * i + 1) * p.br.col_stride) : 1.0f;
      }
    }
  }

  int st = 0;
  for (long long base = first; base < p.M; base += row_step) {
    const long long row = base + slot;
    const bool row_ok = row < p.M;
    {
      int pst = st + STAGES - 1;
      if (pst >= STAGES) pst -= STAGES;
      prefetch(row + (long long)(STAGES - 1) * row_step, pst);
    }
    switch (STAGES) {                             // this row's copies are the oldest group still pending
      case 3: cp_async_wait<2>(); break;
      case 4: cp_async_wait<3>(); break;
      case 5: cp_async_wait<4>(); break;
      case 6: cp_async_wait<5>(); break;
      case 7: cp_async_wait<6>(); break;
      default: cp_async_wait<7>(); break;
    }
    const uint8_t* src = ring + st * stage_bytes + slot * slot_bytes;
    if (++st == STAGES) st = 0;

    float2 x[KMAX][4];
    float rs_res = 1.f, rs_br = 1.f;
    if (row_ok) {
      long long r_res = row, r_br = row;
      if constexpr (EX) { if (p.token_ids) { r_res = table_row(p.token_ids, row, p.n_tok_rows, nullptr); r_br = row % p.seq_len; } }
      if (RES == SRC_I8 && p.res.row_scale) rs_res = __ldg(p.res.row_scale + r_res);
      if (BR == SRC_I8 && p.br.row_scale) rs_br = __ldg(p.br.row_scale + r_br);
    }

    // ---- r = sum of the dequantized addends; running row sum
    float2 s2 = f2(0.f);
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int c = c_first + k * stride;
      if (row_ok && chunk_ok(c)) {
        if constexpr (RES == SRC_I8) {
          const uint2 w = *reinterpret_cast<const uint2*>(src + c * 8);
          i8x8_to_f2(w.x, w.y, x[k]);
          if (p.res.col_scale) {                 // FWQ / SQ residual (the scale is per feature, not per row)
            float2 sc[4];
            if (p.res.col_stride) load_vec8(p.res.col_scale + c * 8, sc);
            else { const float v = __ldg(p.res.col_scale); sc[0] = sc[1] = sc[2] = sc[3] = f2(v); }
#pragma unroll
            for (int i = 0; i < 4; ++i) x[k][i] = __fmul2_rn(x[k][i], sc[i]);
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) x[k][i] = __fmul2_rn(x[k][i], f2(rs_res));
          }
        } else {
          const uint4 w = *reinterpret_cast<const uint4*>(src + c * 16);
          fp16x8_to_f2(w.x, w.y, w.z, w.w, p.res.dt, x[k]);
        }
        if constexpr (BR == SRC_I8) {
          float2 b[4];
          const uint2 wb = *reinterpret_cast<const uint2*>(src + off_br + c * 8);
          i8x8_to_f2(wb.x, wb.y, b);
          if constexpr (CS_REG) {
            if (p.br.row_scale) {
#pragma unroll
              for (int i = 0; i < 4; ++i) x[k][i] = __ffma2_rn(b[i], __fmul2_rn(bcs[k][i], f2(rs_br)), x[k][i]);
            } else {
#pragma unroll
              for (int i = 0; i < 4; ++i) x[k][i] = __ffma2_rn(b[i], bcs[k][i], x[k][i]);
            }
          } else if (p.br.col_scale) {
            float2 sc[4];
            if (p.br.col_stride) load_vec8(p.br.col_scale + c * 8, sc);
            else { const float v = __ldg(p.br.col_scale); sc[0] = sc[1] = sc[2] = sc[3] = f2(v); }
#pragma unroll
            for (int i = 0; i < 4; ++i) x[k][i] = __ffma2_rn(b[i], sc[i], x[k][i]);
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) x[k][i] = __ffma2_rn(b[i], f2(rs_br), x[k][i]);
          }
        }
        if constexpr (BR == SRC_FP) {
          float2 b[4];
          const uint4 wb = *reinterpret_cast<const uint4*>(src + off_br + c * 16);
          fp16x8_to_f2(wb.x, wb.y, wb.z, wb.w, p.br.dt, b);
#pragma unroll
          for (int i = 0; i < 4; ++i) x[k][i] = __fadd2_rn(x[k][i], b[i]);
        }
        if constexpr (EX) {
          float2 e[4];
          const uint4 we = *reinterpret_cast<const uint4*>(src + off_ex + c * 16);
          fp16x8_to_f2(we.x, we.y, we.z, we.w, p.ex.dt, e);
#pragma unroll
          for (int i = 0; i < 4; ++i) x[k][i] = __fadd2_rn(x[k][i], e[i]);
        }
        if constexpr (FPOUT) {
          // the FP residual stream carries the ROUNDED sum; normalise what is stored
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) w[i] = pack_fp2(x[k][i].x, x[k][i].y, p.fp_dt);
          st_global16(reinterpret_cast<char*>(p.fp_out) + (row * p.fp_ld + c * 8) * 2, w[0], w[1], w[2], w[3]);
          fp16x8_to_f2(w[0], w[1], w[2], w[3], p.fp_dt, x[k]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) s2 = __fadd2_rn(s2, x[k][i]);
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) x[k][i] = f2(0.f);
      }
    }
    if constexpr (OUT == O_NONE) continue;

    // ---- mean (true division: a constant row must give exactly zero deviations)
    float s = warp_sum(s2.x + s2.y);
    if (WPR > 1) {
      if (lane == 0) red[0][slot][wr] = s;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "r"(stride) : "memory");
      s = 0.f;
      for (int w = 0; w < WPR; ++w) s += red[0][slot][w];
    }
    const float mean = s / fH;
    // ---- centred (biased) variance over the registers
    float2 q2 = f2(0.f);
    const float2 nm = f2(-mean);
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      if (chunk_ok(c_first + k * stride)) {
#pragma unroll
        for (int i = 0; i < 4; ++i) { x[k][i] = __fadd2_rn(x[k][i], nm); q2 = __ffma2_rn(x[k][i], x[k][i], q2); }
      }
    }
    float q = warp_sum(q2.x + q2.y);
    if (WPR > 1) {
      if (lane == 0) red[1][slot][wr] = q;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "r"(stride) : "memory");
      q = 0.f;
      for (int w = 0; w < WPR; ++w) q += red[1][slot][w];
    }
    const float rstd = rsqrtf(q / fH + p.eps);

    // ---- y = d * (rstd * gamma) + beta ; TWQ: row absmax in the same sweep
    float amax = 0.f;
    const float2 r2 = f2(rstd);
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      const int c = c_first + k * stride;
      if constexpr (GB_REG) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[k][i] = __ffma2_rn(x[k][i], __fmul2_rn(gam[k][i], r2), bet[k][i]);
          if constexpr (OUT == O_TWQ) amax = fmaxf(amax, fmaxf(fabsf(x[k][i].x), fabsf(x[k][i].y)));
        }
      } else if (chunk_ok(c)) {
        float2 g[4], b[4];
        load_vec8(p.gamma + c * 8, g);
        load_vec8(p.beta + c * 8, b);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[k][i] = __ffma2_rn(x[k][i], __fmul2_rn(g[i], r2), b[i]);
          if constexpr (OUT == O_TWQ) amax = fmaxf(amax, fmaxf(fabsf(x[k][i].x), fabsf(x[k][i].y)));
        }
      }
    }

    if constexpr (OUT == O_TWQ) {
      // Eq. 3: S[i] = absmax / 127 on the fly; the scaled value never leaves [-127, 127], so the magic add
      // alone rounds and range-limits it
      amax = warp_max(amax);
      if (WPR > 1) {
        if (lane == 0) red[2][slot][wr] = amax;
        asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "r"(stride) : "memory");
        amax = 0.f;
        for (int w = 0; w < WPR; ++w) amax = fmaxf(amax, red[2][slot][w]);
      }
      const float sc = amax > 0.f ? amax * (1.0f / 127.0f) : 1.0f;
      const float2 inv2 = f2(__fdividef(1.0f, sc)), mg2 = f2(MAGIC);
      if (row_ok && wr == 0 && lane == 0) p.out_scale[row] = sc;
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        const int c = c_first + k * stride;
        if (row_ok && chunk_ok(c)) {
          uint32_t u[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 v = __ffma2_rn(x[k][i], inv2, mg2);
            u[2 * i] = __float_as_uint(v.x); u[2 * i + 1] = __float_as_uint(v.y);
          }
          st_global8(reinterpret_cast<char*>(p.out) + row * p.out_ld + c * 8, pack_low_bytes(u[0], u[1], u[2], u[3]),
                     pack_low_bytes(u[4], u[5], u[6], u[7]));
        }
      }
    } else if constexpr (OUT == O_STATIC) {
      // Eq. 4 / 5: calibrated per-feature (stride 1) or static (stride 0) scale; saturating
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        const int c = c_first + k * stride;
        if (row_ok && chunk_ok(c)) {
          float sc[8];
          if (p.out_gran == HERO_GRAN_FWQ) {
            float4 a = ldg_f4(p.out_scale + c * 8), b = ldg_f4(p.out_scale + c * 8 + 4);
            sc[0] = a.x; sc[1] = a.y; sc[2] = a.z; sc[3] = a.w; sc[4] = b.x; sc[5] = b.y; sc[6] = b.z; sc[7] = b.w;
          } else {
            const float v = __ldg(p.out_scale);
#pragma unroll
            for (int i = 0; i < 8; ++i) sc[i] = v;
          }
          uint32_t u[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float xv = (i & 1) ? x[k][i >> 1].y : x[k][i >> 1].x;
            const float v = fminf(fmaxf(__fdividef(xv, sc[i]), -127.f), 127.f);   // 2 ulp: far below the rounding step
            u[i] = magic_bits(v + MAGIC);
          }
          st_global8(reinterpret_cast<char*>(p.out) + row * p.out_ld + c * 8, pack_low_bytes(u[0], u[1], u[2], u[3]),
                     pack_low_bytes(u[4], u[5], u[6], u[7]));
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < KMAX; ++k) {
        const int c = c_first + k * stride;
        if (row_ok && chunk_ok(c)) {
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) w[i] = pack_fp2(x[k][i].x, x[k][i].y, p.out_dt);
          st_global16(reinterpret_cast<char*>(p.out) + (row * p.out_ld + c * 8) * 2, w[0], w[1], w[2], w[3]);
        }
      }
    }
  }
}

template <int RES, int BR, bool EX, int OUT, bool FPOUT, int NCHX>
static hero_status launch_fast(hero_handle* h, LnParams& p, cudaStream_t stream) {
  const int wpr = p.G;
  const int slots = 8 / wpr;
  const long long want = (p.M + slots - 1) / slots;
  const int es_res = (RES == SRC_I8) ? 1 : 2, es_br = (BR == SRC_I8) ? 1 : (BR == SRC_FP ? 2 : 0);
  const size_t stage = (size_t)slots * p.H * (es_res + es_br + (EX ? 2 : 0));
  // two CTAs per SM; deep enough that about 128 KB per SM are always on their way, within 100 KB per CTA
  int stages = 1 + (int)((64 * 1024 + stage - 1) / stage);
  if (stages < 3) stages = 3;
  if (stages > LNF_MAX_STAGES) stages = LNF_MAX_STAGES;
  while (stages > 3 && stages * stage > 100 * 1024) --stages;
  p.RPC = stages;
  const size_t smem = (size_t)stages * stage;
  auto kern = ln_fast_kernel<RES, BR, EX, OUT, FPOUT, NCHX>;
  HERO_SMEM_OPT_IN(h, kern, 160 * 1024);
  int occ = 1;
  HERO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, LNF_THREADS, smem));
  if (occ < 1) occ = 1;
  const long long cap = (long long)h->sm_count * occ;
  const int grid = (int)(want < cap ? want : cap);
  {
    LaunchScope scope(h, stream, KERNEL_LN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(LNF_THREADS), smem, stream, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

// ------------------------------------------------------------------------------------------------------
// Rows of exactly 1024 * WPR elements (H = 1024, 2048, 4096, 8192): everything a row needs per element is
// decided at compile time.  A lane owns two chunks of 16 consecutive elements (one 16-byte copy per INT8
// chunk, two per FP16 / BF16 chunk), gamma and beta live in registers, the per-feature scale vectors of the
// INT8 addends (and of a static INT8 output) are staged once per CTA in shared memory, and the row loop has
// no parameter-dependent branch.  Same arithmetic, in the same order, as ln_fast_kernel.
//   RES / BR : SRC_I8 | SRC_FP (| SRC_NONE for BR);  RSC: the INT8 residual carries a per-row scale (TWQ,
//   RS_ROW) or a per-feature vector (FWQ / SQ, RS_COL);  an INT8 branch always carries a per-feature vector;
//   BF: the FP tensors involved are BF16 (else FP16);  F8: the 8-bit tensors involved hold e4m3 values instead of INT8
//   (FP8 variant: scale absmax / 448, saturating conversion instead of round + clip).
// ------------------------------------------------------------------------------------------------------
constexpr int RS_ROW = 0, RS_COL = 1;

template <bool BF>
__device__ __forceinline__ void fpx8_to_f2(const uint4 w, float2* v) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if constexpr (BF) v[i] = make_float2(__uint_as_float(u[i] << 16), __uint_as_float(u[i] & 0xffff0000u));
    else v[i] = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
  }
}
template <bool BF>
__device__ __forceinline__ uint32_t pack_fpx2(float a, float b) {
  if constexpr (BF) { __nv_bfloat162 h = __floats2bfloat162_rn(a, b); return *reinterpret_cast<uint32_t*>(&h); }
  else { __half2 h = __floats2half2_rn(a, b); return *reinterpret_cast<uint32_t*>(&h); }
}
__device__ __forceinline__ void i8x16_to_f2(const uint4 w, float2* v) {
  float2 a[4], b[4];
  i8x8_to_f2(w.x, w.y, a);
  i8x8_to_f2(w.z, w.w, b);
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[i] = a[i]; v[4 + i] = b[i]; }
}
// 16 e4m3 bytes -> 8 float pairs (the conversion instruction takes two bytes at a time)
__device__ __forceinline__ void e4m3x16_to_f2(const uint4 w, float2* v) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = ptx::e4m3x2_to_f32x2(u[i] & 0xffffu); v[2 * i + 1] = ptx::e4m3x2_to_f32x2(u[i] >> 16); }
}
template <bool F8>
__device__ __forceinline__ void q8x16_to_f2(const uint4 w, float2* v) {
  if constexpr (F8) e4m3x16_to_f2(w, v); else i8x16_to_f2(w, v);
}
// The CE (16 or 8) floats of one chunk from a piece-major vector in shared memory: piece i of chunk c at float4 index
// i * NCHUNK + c
template <int NCHUNK, int CE>
__device__ __forceinline__ void lds_vec(const float* s, float2* v) {
#pragma unroll
  for (int i = 0; i < CE / 4; ++i) {
    const float4 q = *reinterpret_cast<const float4*>(s + 4 * i * NCHUNK);
    v[2 * i] = make_float2(q.x, q.y); v[2 * i + 1] = make_float2(q.z, q.w);
  }
}
// one chunk of CE 8-bit codes (INT8 or e4m3) / CE FP16-BF16 values from the ring -> CE / 2 float pairs
template <int CE, bool F8>
__device__ __forceinline__ void ring_q8(const uint8_t* src, float2* v) {
  if constexpr (CE == 16) {
    q8x16_to_f2<F8>(*reinterpret_cast<const uint4*>(src), v);
  } else {
    const uint2 w = *reinterpret_cast<const uint2*>(src);
    if constexpr (F8) {
      v[0] = ptx::e4m3x2_to_f32x2(w.x & 0xffffu); v[1] = ptx::e4m3x2_to_f32x2(w.x >> 16);
      v[2] = ptx::e4m3x2_to_f32x2(w.y & 0xffffu); v[3] = ptx::e4m3x2_to_f32x2(w.y >> 16);
    } else {
      float2 t[4];
      i8x8_to_f2(w.x, w.y, t);
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] = t[i];
    }
  }
}
template <int CE, bool BF>
__device__ __forceinline__ void ring_fp(const uint8_t* src, float2* v) {
  fpx8_to_f2<BF>(*reinterpret_cast<const uint4*>(src), v);
  if constexpr (CE == 16) fpx8_to_f2<BF>(*reinterpret_cast<const uint4*>(src + 16), v + 4);
}
// BYTES (8, 16 or 32) of one chunk: global -> ring
template <int BYTES>
__device__ __forceinline__ void copy_chunk(uint8_t* dst, const char* src) {
  if constexpr (BYTES == 8) cp_async8(dst, src);
  else {
    cp_async16(dst, src);
    if constexpr (BYTES == 32) cp_async16(dst + 16, src + 16);
  }
}

// Ring depth of ln_wide_kernel: two CTAs per SM; deep enough that about 128 KB per SM are always on their way,
// within 100 KB per CTA (ring + staged vectors).
__host__ __device__ constexpr int ln_wide_stages(int stage_bytes, int vec_bytes, int wpr, int minb = 2, int least = 3) {
  // (rows of 8192 elements, one per stage, want one stage more: 317 against 334 us on 65536 x 8192 FP16 -> INT8)
  int stages = 1 + ((wpr == 8 ? 80 : 64) * 2 / minb * 1024 + stage_bytes - 1) / stage_bytes;
  if (stages < least) stages = least;
  if (stages > 8) stages = 8;
  while (stages > least && stages * stage_bytes + vec_bytes > 200 / minb * 1024) --stages;
  return stages;
}
// sums / maxima over the LPR consecutive lanes that share a row (32: the warp; 16: a half-warp)
template <int LPR> __device__ __forceinline__ float lanes_sum(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int LPR> __device__ __forceinline__ float lanes_max(float v) {
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// GEO 0: rows of 1024 * WPR elements, WPR >= 2 warps per row, a lane owns two chunks of 16 elements, gamma / beta in
// registers.  Rows of one warp's width are processed two per warp, gamma / beta read from shared memory like the scale
// vectors (the kernel with one row per warp was bound by the shared-memory pipe, 80 % busy, two thirds of its wavefronts
// the FP32 per-column vectors, and by its per-row chain):
// GEO 7: rows of 1024: every lane holds its two chunks of BOTH rows, so a per-column vector is read once for two rows;
// GEO 6: rows of 768: 16 lanes per row, three chunks of 16 per lane (16-byte copies; 32 lanes would need 8-byte ones), the
//        row reductions take four shuffle steps for two rows at once.
template <int RES, int RSC, int BR, int OUT, bool FPOUT, bool BF, int WPR, bool F8, int GEO>
__global__ void __launch_bounds__(LNF_THREADS, 2) ln_wide_kernel(const LnParams p) {
  ptx::pdl_launch_dependents();
  constexpr bool HALF = GEO == 6;                  // two rows per warp, 16 lanes each (WPR = 1): rows of 768
  constexpr bool DUAL = GEO == 7;                  // two rows per warp, every lane holds its columns of both (WPR = 1)
  constexpr int RPL = DUAL ? 2 : 1;                // rows per lane
  static_assert(!HALF || WPR == 1, "half-warp rows are for rows of one warp's width");
  constexpr int LPR = HALF ? 16 : 32;              // lanes that share a row
  static_assert(GEO == 0 || GEO == 6 || GEO == 7, "unknown row geometry");
  static_assert(!DUAL || WPR == 1, "two rows per lane are for rows of one warp's width");
  constexpr int CE = 16;                           // elements per chunk
  constexpr int CPL = HALF ? 3 : 2;                // chunks per lane
  constexpr bool GBS = HALF || DUAL;               // gamma / beta staged in shared memory
  constexpr int MINB = 2;
  constexpr int NP = CE / 2;                       // float pairs per chunk
  constexpr int H = CE * LPR * CPL * WPR;
  constexpr int SLOTS = HALF || DUAL ? 16 : 8 / WPR;   // rows per CTA pass
  constexpr int STRIDE = WPR * LPR;                // chunk stride between a lane's chunks
  constexpr int ES_RES = (RES == SRC_I8) ? 1 : 2;
  constexpr int ES_BR = (BR == SRC_I8) ? 1 : (BR == SRC_FP ? 2 : 0);
  constexpr int OFF_BR = H * ES_RES;
  constexpr int SLOT_BYTES = OFF_BR + H * ES_BR;
  constexpr int STAGE_BYTES = SLOT_BYTES * SLOTS;
  constexpr bool RES_CS = RES == SRC_I8 && RSC == RS_COL;
  constexpr bool BR_CS = BR == SRC_I8;
  constexpr bool OUT_CS = OUT == O_STATIC;
  constexpr int VEC_BYTES = H * 4 * ((RES_CS ? 1 : 0) + (BR_CS ? 1 : 0) + (OUT_CS ? 1 : 0) + (GBS ? 2 : 0));
  constexpr int STAGES = ln_wide_stages(STAGE_BYTES, VEC_BYTES, WPR, MINB, HALF || DUAL ? 2 : 3);   // ring depth
  __shared__ float red[3][8][8];                   // [statistic][row slot][warp in row]
  extern __shared__ __align__(16) uint8_t dyn[];
  float* v_rcs = reinterpret_cast<float*>(dyn);
  float* v_bcs = v_rcs + (RES_CS ? H : 0);
  float* v_ocs = v_bcs + (BR_CS ? H : 0);
  float* v_gam = v_ocs + (OUT_CS ? H : 0);
  float* v_bet = v_gam + (GBS ? H : 0);
  uint8_t* ring = reinterpret_cast<uint8_t*>(v_bet + (GBS ? H : 0));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slot = HALF ? warp * 2 + (lane >> 4) : (DUAL ? warp * 2 : warp / WPR), wr = HALF || DUAL ? 0 : warp % WPR;
  const int hl = lane & (LPR - 1);                 // this lane's position among the lanes of its row
  const int c_first = wr * 32 + hl;                // this lane's first chunk (16-element units)
  const float MAGIC = 12582912.0f;                 // 1.5 * 2^23
  constexpr float fH = (float)H;

  const char* g_res = reinterpret_cast<const char*>(p.res.data) + c_first * CE * ES_RES;
  const char* g_br = (BR != SRC_NONE) ? reinterpret_cast<const char*>(p.br.data) + c_first * CE * ES_BR : nullptr;
  const long long pitch_res = p.res.ld * ES_RES, pitch_br = (BR != SRC_NONE) ? p.br.ld * ES_BR : 0;
  uint8_t* my_ring = ring + slot * SLOT_BYTES + c_first * CE * ES_RES;          // residual part of this lane's slice
  uint8_t* my_ring_br = ring + slot * SLOT_BYTES + OFF_BR + c_first * CE * ES_BR;

  // A lane copies exactly the chunks it will later read, so waiting on its own copy groups is all the
  // synchronisation the ring needs.
  auto prefetch = [&](long long row0, int st) {
#pragma unroll
    for (int u = 0; u < RPL; ++u) {
      const long long row = row0 + u;              // (two rows per lane: consecutive rows, consecutive ring slots)
      if (row < p.M) {                             // rows past the end still commit an (empty) group
        const char* gr = g_res + row * pitch_res;
        uint8_t* d = my_ring + st * STAGE_BYTES + u * SLOT_BYTES;
#pragma unroll
        for (int k = 0; k < CPL; ++k) copy_chunk<CE * ES_RES>(d + k * STRIDE * CE * ES_RES, gr + k * STRIDE * CE * ES_RES);
        if constexpr (BR != SRC_NONE) {
          const char* gb = g_br + row * pitch_br;
          uint8_t* db = my_ring_br + st * STAGE_BYTES + u * SLOT_BYTES;
#pragma unroll
          for (int k = 0; k < CPL; ++k) copy_chunk<CE * ES_BR>(db + k * STRIDE * CE * ES_BR, gb + k * STRIDE * CE * ES_BR);
        }
      }
    }
    cp_async_commit();
  };

  // Everything that does not depend on the previous kernel comes first (calibrated scale vectors, gamma, beta): with a
  // programmatic dependent launch it overlaps that kernel's tail.
  // per-feature vectors: shared memory for the scales, registers for gamma / beta
  // stored piece-major ([float4 piece q of a chunk][chunk]): consecutive lanes then read consecutive 16-byte words,
  // free of bank conflicts
  for (int i = threadIdx.x; i < H; i += LNF_THREADS) {
    const int si = ((((i % CE) >> 2) * (H / CE)) + i / CE) * 4 + (i & 3);
    if constexpr (RES_CS) v_rcs[si] = __ldg(p.res.col_scale + i * p.res.col_stride);
    if constexpr (BR_CS) v_bcs[si] = __ldg(p.br.col_scale + i * p.br.col_stride);
    if constexpr (OUT_CS) v_ocs[si] = 1.0f / __ldg(p.out_scale + (p.out_gran == HERO_GRAN_FWQ ? i : 0));   // reciprocal, see the output stage
    if constexpr (GBS && OUT != O_NONE) { v_gam[si] = __ldg(p.gamma + i); v_bet[si] = __ldg(p.beta + i); }
  }
  float2 gam[GBS ? 1 : CPL][NP], bet[GBS ? 1 : CPL][NP];
  if constexpr (OUT != O_NONE && !GBS) {
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
      const int e0 = (c_first + k * STRIDE) * CE;
#pragma unroll
      for (int j = 0; j < CE / 8; ++j) {
        float2 t[4];
        load_vec8(p.gamma + e0 + 8 * j, t);
#pragma unroll
        for (int i = 0; i < 4; ++i) gam[k][4 * j + i] = t[i];
        load_vec8(p.beta + e0 + 8 * j, t);
#pragma unroll
        for (int i = 0; i < 4; ++i) bet[k][4 * j + i] = t[i];
      }
    }
  }
  ptx::pdl_wait();                                 // the previous kernel's outputs are complete and visible from here on
  const long long row_step = (long long)gridDim.x * SLOTS;
  const long long first = (long long)blockIdx.x * SLOTS + slot;
  for (int s0 = 0; s0 < STAGES - 1; ++s0) prefetch(first + s0 * row_step, s0);
  // the per-row scale of a TWQ residual travels STAGES - 1 rows ahead as well, in a register ring: lane i of a warp
  // holds the scale of the i-th row ahead (STAGES <= 8 < 32)
  constexpr bool ROW_SC = RES == SRC_I8 && RSC == RS_ROW;
  float rs_ring[RPL];
#pragma unroll
  for (int u = 0; u < RPL; ++u) {
    rs_ring[u] = 1.f;
    if constexpr (ROW_SC) {
      const long long r = first + u + (long long)hl * row_step;
      if (hl < STAGES - 1 && r < p.M) rs_ring[u] = __ldg(p.res.row_scale + r);
    }
  }

  __syncthreads();

  int st = 0;
  // every slot walks its own rows: nothing in the loop is shared between slots (named barriers are per slot)
  // (half-warp rows: the warp's two rows are consecutive, so the loop runs while the lower one exists and the upper half
  // computes on stale ring contents, stores nothing, on the last pass of an odd tail; shuffles never cross the halves)
  // (two rows per lane: a lane holds its columns of the warp's two rows, so every per-column vector is read once for both)
  for (long long row = first; row - (HALF ? (lane >> 4) : 0) < p.M; row += row_step) {
    bool row_in[RPL];
#pragma unroll
    for (int u = 0; u < RPL; ++u) row_in[u] = !(HALF || DUAL) || row + u < p.M;
    {
      int pst = st + STAGES - 1;
      if (pst >= STAGES) pst -= STAGES;
      prefetch(row + (long long)(STAGES - 1) * row_step, pst);
    }
    float rs_res[RPL];
#pragma unroll
    for (int u = 0; u < RPL; ++u) {
      rs_res[u] = 1.f;
      if constexpr (ROW_SC) {
        // this row's scale sits in lane 0; shift the ring by one lane and let lane STAGES - 2 fetch the newest row's
        rs_res[u] = __shfl_sync(0xffffffffu, rs_ring[u], 0, LPR);
        rs_ring[u] = __shfl_down_sync(0xffffffffu, rs_ring[u], 1, LPR);
        const long long r = row + u + (long long)(STAGES - 1) * row_step;
        if (hl == STAGES - 2 && r < p.M) rs_ring[u] = __ldg(p.res.row_scale + r);
      }
    }
    cp_async_wait<STAGES - 1>();                   // this row's copies are the oldest group still pending
    const uint8_t* src = my_ring + st * STAGE_BYTES;
    const uint8_t* src_br = my_ring_br + st * STAGE_BYTES;
    if (++st == STAGES) st = 0;

    // ---- r = sum of the dequantized addends; running row sum
    float2 x[RPL][CPL][NP];
    float2 s2[RPL];
#pragma unroll
    for (int u = 0; u < RPL; ++u) s2[u] = f2(0.f);
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
      float2 rcs[RES_CS ? NP : 1], bcs[BR_CS ? NP : 1];
      if constexpr (RES_CS) lds_vec<H / CE, CE>(v_rcs + (c_first + k * STRIDE) * 4, rcs);
      if constexpr (BR_CS) lds_vec<H / CE, CE>(v_bcs + (c_first + k * STRIDE) * 4, bcs);
#pragma unroll
      for (int u = 0; u < RPL; ++u) {
        if constexpr (RES == SRC_I8) {
          ring_q8<CE, F8>(src + u * SLOT_BYTES + k * STRIDE * CE, x[u][k]);
          if constexpr (RSC == RS_COL) {
#pragma unroll
            for (int i = 0; i < NP; ++i) x[u][k][i] = __fmul2_rn(x[u][k][i], rcs[i]);
          } else {
#pragma unroll
            for (int i = 0; i < NP; ++i) x[u][k][i] = __fmul2_rn(x[u][k][i], f2(rs_res[u]));
          }
        } else {
          ring_fp<CE, BF>(src + u * SLOT_BYTES + k * STRIDE * CE * 2, x[u][k]);
        }
        if constexpr (BR == SRC_I8) {
          float2 b[NP];
          ring_q8<CE, F8>(src_br + u * SLOT_BYTES + k * STRIDE * CE, b);
#pragma unroll
          for (int i = 0; i < NP; ++i) x[u][k][i] = __ffma2_rn(b[i], bcs[i], x[u][k][i]);
        }
        if constexpr (BR == SRC_FP) {
          float2 b[NP];
          ring_fp<CE, BF>(src_br + u * SLOT_BYTES + k * STRIDE * CE * 2, b);
#pragma unroll
          for (int i = 0; i < NP; ++i) x[u][k][i] = __fadd2_rn(x[u][k][i], b[i]);
        }
        if constexpr (FPOUT) {
          // the FP residual stream carries the ROUNDED sum; normalise what is stored
          uint32_t w[NP];
#pragma unroll
          for (int i = 0; i < NP; ++i) w[i] = pack_fpx2<BF>(x[u][k][i].x, x[u][k][i].y);
          char* dst = reinterpret_cast<char*>(p.fp_out) + ((row + u) * p.fp_ld + (c_first + k * STRIDE) * CE) * 2;
#pragma unroll
          for (int j = 0; j < CE / 8; ++j) {
            if (row_in[u]) st_global16(dst + 16 * j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            fpx8_to_f2<BF>(make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]), x[u][k] + 4 * j);
          }
        }
#pragma unroll
        for (int i = 0; i < NP; ++i) s2[u] = __fadd2_rn(s2[u], x[u][k][i]);
      }
    }
    if constexpr (OUT == O_NONE) continue;

    // ---- mean (true division: a constant row must give exactly zero deviations), then the centred (biased) variance
    float rstd[RPL];
#pragma unroll
    for (int u = 0; u < RPL; ++u) {
      float s = lanes_sum<LPR>(s2[u].x + s2[u].y);
      if constexpr (WPR > 1) {
        if (lane == 0) red[0][slot][wr] = s;
        asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "n"(STRIDE) : "memory");
        s = 0.f;
#pragma unroll
        for (int w = 0; w < WPR; ++w) s += red[0][slot][w];
      }
      const float mean = s / fH;
      float2 q2 = f2(0.f);
      const float2 nm = f2(-mean);
#pragma unroll
      for (int k = 0; k < CPL; ++k) {
#pragma unroll
        for (int i = 0; i < NP; ++i) { x[u][k][i] = __fadd2_rn(x[u][k][i], nm); q2 = __ffma2_rn(x[u][k][i], x[u][k][i], q2); }
      }
      float q = lanes_sum<LPR>(q2.x + q2.y);
      if constexpr (WPR > 1) {
        if (lane == 0) red[1][slot][wr] = q;
        asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "n"(STRIDE) : "memory");
        q = 0.f;
#pragma unroll
        for (int w = 0; w < WPR; ++w) q += red[1][slot][w];
      }
      rstd[u] = rsqrtf(q / fH + p.eps);            // 2 ulp: far below the rounding step of the output
    }

    // ---- y = d * (rstd * gamma) + beta ; TWQ: row absmax in the same sweep
    float amax[RPL];
#pragma unroll
    for (int u = 0; u < RPL; ++u) amax[u] = 0.f;
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
      if constexpr (GBS) {
        lds_vec<H / CE, CE>(v_gam + (c_first + k * STRIDE) * 4, gam[0]);
        lds_vec<H / CE, CE>(v_bet + (c_first + k * STRIDE) * 4, bet[0]);
      }
#pragma unroll
      for (int u = 0; u < RPL; ++u) {
        const float2 r2 = f2(rstd[u]);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          x[u][k][i] = __ffma2_rn(x[u][k][i], __fmul2_rn(gam[GBS ? 0 : k][i], r2), bet[GBS ? 0 : k][i]);
          if constexpr (OUT == O_TWQ) amax[u] = fmaxf(amax[u], fmaxf(fabsf(x[u][k][i].x), fabsf(x[u][k][i].y)));
        }
      }
    }

    if constexpr (OUT == O_TWQ) {
      // Eq. 3: S[i] = absmax / 127 on the fly; the scaled value never leaves [-127, 127], so the magic add
      // alone rounds and range-limits it
#pragma unroll
      for (int u = 0; u < RPL; ++u) {
        float am = lanes_max<LPR>(amax[u]);
        if constexpr (WPR > 1) {
          if (lane == 0) red[2][slot][wr] = am;
          asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "n"(STRIDE) : "memory");
          am = 0.f;
#pragma unroll
          for (int w = 0; w < WPR; ++w) am = fmaxf(am, red[2][slot][w]);
        }
        const float sc = am > 0.f ? am * (F8 ? 1.0f / 448.0f : 1.0f / 127.0f) : 1.0f;   // within 1 ulp of the quotient
        const float2 inv2 = f2(__fdividef(1.0f, sc)), mg2 = f2(MAGIC);
        if (wr == 0 && hl == 0 && row_in[u]) p.out_scale[row + u] = sc;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
          uint32_t w[CE / 4];
#pragma unroll
          for (int g = 0; g < CE / 4; ++g) {
            if constexpr (F8) {
              const float2 a = __fmul2_rn(x[u][k][2 * g], inv2), b = __fmul2_rn(x[u][k][2 * g + 1], inv2);
              w[g] = ptx::f32x4_to_e4m3x4(a.x, a.y, b.x, b.y);
            } else {
              const float2 a = __ffma2_rn(x[u][k][2 * g], inv2, mg2), b = __ffma2_rn(x[u][k][2 * g + 1], inv2, mg2);
              w[g] = pack_low_bytes(__float_as_uint(a.x), __float_as_uint(a.y), __float_as_uint(b.x), __float_as_uint(b.y));
            }
          }
          char* dst = reinterpret_cast<char*>(p.out) + (row + u) * p.out_ld + (c_first + k * STRIDE) * CE;
          if (row_in[u]) {
            if constexpr (CE == 16) st_global16(dst, w[0], w[1], w[2], w[3]);
            else st_global8(dst, w[0], w[1]);
          }
        }
      }
    } else if constexpr (OUT == O_STATIC) {
      // Eq. 4 / 5: calibrated per-feature or static scale, saturating.  The staged vector holds the reciprocals (one true
      // division per feature and CTA): the product is within one ulp of the quotient
      {
        const float2 lo2 = f2(-127.f), hi2 = f2(127.f), mg2 = f2(MAGIC);
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
          float2 sc[NP];
          lds_vec<H / CE, CE>(v_ocs + (c_first + k * STRIDE) * 4, sc);
#pragma unroll
          for (int u = 0; u < RPL; ++u) {
            uint32_t w[CE / 4];
#pragma unroll
            for (int g = 0; g < CE / 4; ++g) {
              const float2 a = __fmul2_rn(x[u][k][2 * g], sc[2 * g]), b = __fmul2_rn(x[u][k][2 * g + 1], sc[2 * g + 1]);
              if constexpr (F8) {
                w[g] = ptx::f32x4_to_e4m3x4(a.x, a.y, b.x, b.y);
              } else {
                const float a0 = fminf(fmaxf(a.x, lo2.x), hi2.x) + mg2.x, a1 = fminf(fmaxf(a.y, lo2.x), hi2.x) + mg2.x;
                const float b0 = fminf(fmaxf(b.x, lo2.x), hi2.x) + mg2.x, b1 = fminf(fmaxf(b.y, lo2.x), hi2.x) + mg2.x;
                w[g] = pack_low_bytes(__float_as_uint(a0), __float_as_uint(a1), __float_as_uint(b0), __float_as_uint(b1));
              }
            }
            char* dst = reinterpret_cast<char*>(p.out) + (row + u) * p.out_ld + (c_first + k * STRIDE) * CE;
            if (row_in[u]) {
              if constexpr (CE == 16) st_global16(dst, w[0], w[1], w[2], w[3]);
              else st_global8(dst, w[0], w[1]);
            }
          }
        }
      }
    } else {
      {
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
#pragma unroll
          for (int u = 0; u < RPL; ++u) {
            uint32_t w[NP];
#pragma unroll
            for (int i = 0; i < NP; ++i) w[i] = pack_fpx2<BF>(x[u][k][i].x, x[u][k][i].y);
            char* dst = reinterpret_cast<char*>(p.out) + ((row + u) * p.out_ld + (c_first + k * STRIDE) * CE) * 2;
#pragma unroll
            for (int j = 0; j < CE / 8; ++j) if (row_in[u]) st_global16(dst + 16 * j, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
          }
        }
      }
    }
  }
  cp_async_wait<0>();
}

template <int RES, int RSC, int BR, int OUT, bool FPOUT, bool BF, int WPR, bool F8, int GEO>
static hero_status launch_wide(hero_handle* h, LnParams& p, cudaStream_t stream) {
  constexpr int H = (GEO == 6 ? 768 : 1024) * WPR, SLOTS = GEO >= 6 ? 16 : 8 / WPR;   // (GEO 6, 7: two rows per warp)
  constexpr int ES_RES = (RES == SRC_I8) ? 1 : 2, ES_BR = (BR == SRC_I8) ? 1 : (BR == SRC_FP ? 2 : 0);
  constexpr size_t STAGE = (size_t)SLOTS * H * (ES_RES + ES_BR);
  constexpr size_t VEC = (size_t)H * 4 * ((RES == SRC_I8 && RSC == RS_COL ? 1 : 0) + (BR == SRC_I8 ? 1 : 0) + (OUT == O_STATIC ? 1 : 0) + (GEO >= 6 ? 2 : 0));
  constexpr int stages = ln_wide_stages((int)STAGE, (int)VEC, WPR, 2, GEO >= 6 ? 2 : 3);
  const size_t smem = (size_t)stages * STAGE + VEC;
  auto kern = ln_wide_kernel<RES, RSC, BR, OUT, FPOUT, BF, WPR, F8, GEO>;
  HERO_SMEM_OPT_IN(h, kern, 200 * 1024);
  static PerDeviceInt occ_cache;     // per instantiation and device: the launch configuration never changes
  int occ = occ_cache.get(h->device);
  if (occ < 1) {
    HERO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, LNF_THREADS, smem));
    if (occ < 1) occ = 1;
    occ_cache.set(h->device, occ);
  }
  const long long want = (p.M + SLOTS - 1) / SLOTS;
  const long long cap = (long long)h->sm_count * occ;
  const int grid = (int)(want < cap ? want : cap);
  {
    LaunchScope scope(h, stream, KERNEL_LN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(LNF_THREADS), smem, stream, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

template <int RES, int RSC, int BR, int OUT, bool FPOUT, bool BF, bool F8>
static hero_status launch_wide_wpr(hero_handle* h, LnParams& p, cudaStream_t s) {
  switch (p.H) {
    case 768: return launch_wide<RES, RSC, BR, OUT, FPOUT, BF, 1, F8, 6>(h, p, s);
    case 1024: return launch_wide<RES, RSC, BR, OUT, FPOUT, BF, 1, F8, 7>(h, p, s);
    case 2048: return launch_wide<RES, RSC, BR, OUT, FPOUT, BF, 2, F8, 0>(h, p, s);
    case 4096: return launch_wide<RES, RSC, BR, OUT, FPOUT, BF, 4, F8, 0>(h, p, s);
    default: return launch_wide<RES, RSC, BR, OUT, FPOUT, BF, 8, F8, 0>(h, p, s);
  }
}

// The combinations the layer forward produces on rows of 1024 * {1, 2, 4, 8} elements.
static hero_status try_wide(hero_handle* h, LnParams& p, cudaStream_t s, bool* taken) {
  *taken = false;
  if (!(p.H == 768 || p.H == 1024 || p.H == 2048 || p.H == 4096 || p.H == 8192) || p.ex.data || p.token_ids) return HERO_OK;
  // one 8-bit payload across the call (INT8, or e4m3 for the FP8 variant); a mix takes the generic kernel
  int q8t = -1;
  auto q8_ok = [&](bool used, int dt) { if (!used || !is_q8(dt)) return true; if (q8t < 0) q8t = dt; return q8t == dt; };
  if (!q8_ok(true, p.res.dt) || !q8_ok(p.br.data != nullptr, p.br.dt) || !q8_ok(p.out != nullptr, p.out_dt)) return HERO_OK;
  const bool f8 = q8t == HERO_F8;
  const int res = is_q8(p.res.dt) ? SRC_I8 : SRC_FP;
  const int br = !p.br.data ? SRC_NONE : (is_q8(p.br.dt) ? SRC_I8 : SRC_FP);
  const int out = !p.out ? O_NONE : (!is_q8(p.out_dt) ? O_FP : (p.out_gran == HERO_GRAN_TWQ ? O_TWQ : O_STATIC));
  const bool fpo = p.fp_out != nullptr;
  // scale kinds the kernel is specialised for
  int rsc = RS_ROW;
  if (res == SRC_I8) {
    if (p.res.row_scale && !p.res.col_scale) rsc = RS_ROW;
    else if (!p.res.row_scale && p.res.col_scale) rsc = RS_COL;
    else return HERO_OK;
  }
  if (br == SRC_I8 && (p.br.row_scale || !p.br.col_scale)) return HERO_OK;
  if (out == O_STATIC && !(p.out_gran == HERO_GRAN_FWQ || p.out_gran == HERO_GRAN_SQ)) return HERO_OK;
  // one FP type across the call
  int fpt = -1;
  auto fp_ok = [&](bool used, int dt) { if (!used) return true; if (fpt < 0) fpt = dt; return fpt == dt; };
  if (!fp_ok(res == SRC_FP, p.res.dt) || !fp_ok(br == SRC_FP, p.br.dt) || !fp_ok(out == O_FP, p.out_dt) || !fp_ok(fpo, p.fp_dt))
    return HERO_OK;
  const bool bf = fpt == HERO_BF16;
#define LNW_CASE(R_, S_, B_, O_, F_)                                                                 \
  if (res == R_ && (R_ != SRC_I8 || rsc == S_) && br == B_ && out == O_ && fpo == F_) {               \
    *taken = true;                                                                                   \
    if (f8) return bf ? launch_wide_wpr<R_, S_, B_, O_, F_, true, true>(h, p, s) : launch_wide_wpr<R_, S_, B_, O_, F_, false, true>(h, p, s); \
    return bf ? launch_wide_wpr<R_, S_, B_, O_, F_, true, false>(h, p, s) : launch_wide_wpr<R_, S_, B_, O_, F_, false, false>(h, p, s); \
  }
  LNW_CASE(SRC_I8, RS_COL, SRC_I8, O_TWQ, false)      // Eq. 19: FWQ / SQ residual + FWQ branch -> TWQ
  LNW_CASE(SRC_I8, RS_ROW, SRC_I8, O_TWQ, false)      // Eq. 31: TWQ residual + FWQ branch -> TWQ
  LNW_CASE(SRC_I8, RS_COL, SRC_I8, O_STATIC, false)
  LNW_CASE(SRC_I8, RS_ROW, SRC_I8, O_STATIC, false)
  LNW_CASE(SRC_I8, RS_COL, SRC_I8, O_FP, false)
  LNW_CASE(SRC_I8, RS_ROW, SRC_I8, O_FP, false)
  LNW_CASE(SRC_FP, RS_ROW, SRC_NONE, O_TWQ, false)    // entry LN^quant / pre-LN LN1
  LNW_CASE(SRC_FP, RS_ROW, SRC_NONE, O_STATIC, false)
  LNW_CASE(SRC_FP, RS_ROW, SRC_I8, O_TWQ, true)       // pre-LN: add + LN + quant, new residual stream stored
  LNW_CASE(SRC_FP, RS_ROW, SRC_I8, O_STATIC, true)
  LNW_CASE(SRC_FP, RS_ROW, SRC_I8, O_NONE, true)      // closing residual add of a lone pre-LN layer
#undef LNW_CASE
  // modules left in FP16 / BF16 (Table 1): no 8-bit tensor in the call
#define LNW_FP_CASE(B_, O_, F_)                                                                       \
  if (res == SRC_FP && br == B_ && out == O_ && fpo == F_) {                                            \
    *taken = true;                                                                                   \
    return bf ? launch_wide_wpr<SRC_FP, RS_ROW, B_, O_, F_, true, false>(h, p, s)                       \
              : launch_wide_wpr<SRC_FP, RS_ROW, B_, O_, F_, false, false>(h, p, s);                     \
  }
  LNW_FP_CASE(SRC_FP, O_FP, false)                    // post-LN: residual + branch -> FP
  LNW_FP_CASE(SRC_NONE, O_FP, false)                  // pre-LN LN1 feeding an FP QKV
  LNW_FP_CASE(SRC_FP, O_FP, true)                     // pre-LN: add + LN, new residual stream stored
  LNW_FP_CASE(SRC_FP, O_NONE, true)                   // closing residual add
#undef LNW_FP_CASE
  return HERO_OK;
}

// Returns HERO_ERR_UNSUPPORTED (without setting an error) when the combination has no fast instantiation.
static hero_status try_fast(hero_handle* h, LnParams& p, cudaStream_t s, bool* taken) {
  *taken = false;
  if (p.H % 8 != 0 || p.H > 8192) return HERO_OK;
  if (p.res.dt == HERO_F8 || (p.br.data && p.br.dt == HERO_F8) || (p.out && p.out_dt == HERO_F8)) return HERO_OK;   // generic kernel
  const int res = p.res.dt == HERO_I8 ? SRC_I8 : SRC_FP;
  const int br = !p.br.data ? SRC_NONE : (p.br.dt == HERO_I8 ? SRC_I8 : SRC_FP);
  const bool ex = p.ex.data != nullptr;
  const int out = !p.out ? O_NONE : (p.out_dt != HERO_I8 ? O_FP : (p.out_gran == HERO_GRAN_TWQ ? O_TWQ : O_STATIC));
  const bool fpo = p.fp_out != nullptr;
  if (res == SRC_I8 && p.res.row_scale && p.res.col_scale) return HERO_OK;
  // rows of exactly 3 or 4 chunks per lane (H = 768, 1024, 4096, 8192, ...) take the tail-free instantiation
  int wpr = 1, exact = 0;
  for (int n = 4; n >= 2 && !exact; --n)              // H = 256 * n * wpr with wpr in {1, 2, 4, 8}
    for (int w = 1; w <= 8 && !exact; w *= 2)
      if (p.H == 256 * n * w) { wpr = w; exact = n; }
  if (!exact) while (wpr * 1024 < p.H) wpr *= 2;
  p.G = wpr;
#define LNF_CASE(R_, B_, E_, O_, F_)                                                   \
  if (res == R_ && br == B_ && ex == E_ && out == O_ && fpo == F_) {                   \
    *taken = true;                                                                     \
    return launch_fast<R_, B_, E_, O_, F_, 0>(h, p, s);                                \
  }
#define LNF_CASE_X(R_, B_, E_, O_, F_)                                                 \
  if (res == R_ && br == B_ && ex == E_ && out == O_ && fpo == F_) {                   \
    *taken = true;                                                                     \
    if (exact == 2) return launch_fast<R_, B_, E_, O_, F_, 2>(h, p, s);                \
    if (exact == 3) return launch_fast<R_, B_, E_, O_, F_, 3>(h, p, s);                \
    if (exact == 4) return launch_fast<R_, B_, E_, O_, F_, 4>(h, p, s);                \
    return launch_fast<R_, B_, E_, O_, F_, 0>(h, p, s);                                \
  }
#define LNF_OUTS(R_, B_, E_, F_) LNF_CASE_X(R_, B_, E_, O_TWQ, F_) LNF_CASE(R_, B_, E_, O_STATIC, F_) LNF_CASE(R_, B_, E_, O_FP, F_)
  LNF_OUTS(SRC_FP, SRC_NONE, false, false)   // entry LN^quant on FP activations; pre-LN LN1
  LNF_OUTS(SRC_I8, SRC_I8, false, false)     // Eq. 19 / 31: two INT8 addends
  LNF_OUTS(SRC_I8, SRC_FP, false, false)     // INT8 residual + FP branch (modes M1 / M2)
  LNF_OUTS(SRC_FP, SRC_FP, false, false)     // all-FP modules
  LNF_OUTS(SRC_FP, SRC_I8, false, false)     // FP residual + INT8 branch
  LNF_OUTS(SRC_FP, SRC_I8, false, true)      // pre-LN: add + LN + quant, new residual stream stored
  LNF_OUTS(SRC_FP, SRC_FP, false, true)
  LNF_CASE_X(SRC_FP, SRC_I8, false, O_NONE, true)   // closing residual add of a lone pre-LN layer
  LNF_CASE(SRC_FP, SRC_FP, false, O_NONE, true)
  LNF_OUTS(SRC_I8, SRC_FP, true, false)      // Eq. 7: embedding gather, three addends
#undef LNF_OUTS
#undef LNF_CASE_X
#undef LNF_CASE
  return HERO_OK;
}

}  // namespace hero

extern "C" hero_status hero_layernorm_quant(hero_handle* h, const hero_ln_args* a, void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && a, HERO_ERR_INVALID_ARG, "hero_layernorm_quant: NULL handle or args");
  LnParams p;
  memset(&p, 0, sizeof(p));
  const bool gather = a->token_ids != nullptr;
  HERO_REQUIRE(a->residual.data != nullptr || (!gather && a->residual.rows == 0), HERO_ERR_INVALID_ARG, "residual is required");
  if (!gather && a->residual.rows == 0) return HERO_OK;
  const int H = (int)a->residual.cols;
  HERO_REQUIRE(H > 0 && H % 16 == 0 && H <= 16384, HERO_ERR_UNSUPPORTED, "H=%d must be a multiple of 16, at most 16384", H);
  hero_status st;
  if ((st = fill_side(a->residual, &p.res, "residual", true, H)) != HERO_OK) return st;
  if ((st = fill_side(a->branch, &p.br, "branch", true, H)) != HERO_OK) return st;
  if ((st = fill_side(a->extra, &p.ex, "extra", false, H)) != HERO_OK) return st;
  p.M = gather ? a->n_tokens : a->residual.rows;
  HERO_REQUIRE(p.M >= 0, HERO_ERR_INVALID_ARG, "negative row count");
  if (gather) {
    HERO_REQUIRE(a->residual.dtype == HERO_I8 && a->residual.gran == HERO_GRAN_TWQ, HERO_ERR_UNSUPPORTED,
                 "embedding gather: the token table must be INT8 with one scale per row (Eq. 7)");
    HERO_REQUIRE(a->seq_len > 0, HERO_ERR_INVALID_ARG, "embedding gather: seq_len must be positive");
    HERO_REQUIRE(a->extra.data == nullptr || a->type_ids != nullptr, HERO_ERR_INVALID_ARG,
                 "embedding gather: type_ids required with a sentence-type table");
    HERO_REQUIRE(a->residual.rows > 0 && a->residual.rows < (1ll << 31), HERO_ERR_INVALID_ARG, "embedding gather: the token table needs 1 .. 2^31-1 rows");
    HERO_REQUIRE(a->branch.data == nullptr || a->branch.rows >= a->seq_len, HERO_ERR_INVALID_ARG,
                 "embedding gather: the position table has %lld rows, seq_len is %d", (long long)a->branch.rows, a->seq_len);
    HERO_REQUIRE(a->extra.data == nullptr || (a->extra.rows > 0 && a->extra.rows < (1ll << 31)), HERO_ERR_INVALID_ARG,
                 "embedding gather: the sentence-type table needs at least one row");
    p.token_ids = a->token_ids; p.type_ids = a->type_ids; p.seq_len = a->seq_len;
    p.n_tok_rows = (int)a->residual.rows; p.n_type_rows = a->extra.data ? (int)a->extra.rows : 1;
    p.err = h->d_error;
  } else {
    HERO_REQUIRE(a->branch.data == nullptr || a->branch.rows == p.M, HERO_ERR_INVALID_ARG, "branch rows differ");
    HERO_REQUIRE(a->extra.data == nullptr || a->extra.rows == p.M, HERO_ERR_INVALID_ARG, "extra rows differ");
    HERO_REQUIRE(a->extra.data == nullptr || a->branch.data != nullptr, HERO_ERR_INVALID_ARG,
                 "extra (third addend) given without branch (second addend)");
  }
  p.H = H;
  p.gamma = a->gamma; p.beta = a->beta; p.eps = a->eps;
  if (a->out.data) {
    if ((st = check_matrix(a->out, "out")) != HERO_OK) return st;
    HERO_REQUIRE(a->gamma && a->beta, HERO_ERR_INVALID_ARG, "gamma and beta are required");
    HERO_REQUIRE(aligned16(a->gamma) && aligned16(a->beta), HERO_ERR_ALIGNMENT, "gamma/beta must be 16-byte aligned");
    HERO_REQUIRE(a->out.rows == p.M && a->out.cols == H, HERO_ERR_INVALID_ARG, "out shape mismatch");
    HERO_REQUIRE(is_q8(a->out.dtype) || is_fp16ish(a->out.dtype), HERO_ERR_UNSUPPORTED, "out dtype %d", a->out.dtype);
    if (is_q8(a->out.dtype))
      HERO_REQUIRE(a->out.gran == HERO_GRAN_TWQ || a->out.gran == HERO_GRAN_FWQ || a->out.gran == HERO_GRAN_SQ,
                   HERO_ERR_INVALID_ARG, "an 8-bit out needs granularity TWQ, FWQ or SQ");
    p.out = a->out.data; p.out_dt = a->out.dtype; p.out_ld = a->out.ld; p.out_gran = a->out.gran;
    p.out_scale = a->out.scale;
  }
  if (a->fp_out.data) {
    if ((st = check_matrix(a->fp_out, "fp_out")) != HERO_OK) return st;
    HERO_REQUIRE(is_fp16ish(a->fp_out.dtype), HERO_ERR_UNSUPPORTED, "fp_out must be F16 or BF16");
    HERO_REQUIRE(a->fp_out.rows == p.M && a->fp_out.cols == H, HERO_ERR_INVALID_ARG, "fp_out shape mismatch");
    p.fp_out = a->fp_out.data; p.fp_dt = a->fp_out.dtype; p.fp_ld = a->fp_out.ld;
  }
  HERO_REQUIRE(p.out || p.fp_out, HERO_ERR_INVALID_ARG, "neither out nor fp_out given");
  if (a->out_col_absmax) {
    HERO_REQUIRE(p.out ? is_fp16ish(p.out_dt) : true, HERO_ERR_UNSUPPORTED,
                 "out_col_absmax observes an F16 / BF16 out (or fp_out when out is absent), not 8-bit codes");
    p.obs = a->out_col_absmax;
  }
  if (p.M == 0) return HERO_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  bool taken = false;
  if (!p.obs) {             // the observer lives in the generic kernel only (calibration is an offline pass)
    st = try_wide(h, p, s, &taken);
    if (taken || st != HERO_OK) return st;
    st = try_fast(h, p, s, &taken);
    if (taken || st != HERO_OK) return st;
  }
  // generic kernel for the remaining combinations.
  // 16 elements per thread when rows are long (fewer, fatter threads); 8 otherwise.  VEC=16 needs H % 16 == 0.
  if (H % 16 == 0 && H >= 2048) return launch_ln<16, 1>(h, p, s);
  return launch_ln<8, 2>(h, p, s);
}

