// One decode step of the INT8 attention core (Sec. 2.2.2 Eq. 15-17 for a single query row per sequence) over an INT8
// key / value cache.  The step reads every cached key and value once and does two operations per byte: what bounds it
// is HBM bandwidth, so the kernel is built around wide coalesced loads and enough of them in flight, not around the
// tensor cores (a 1-row product would use 1/128 of an MMA tile).
//
// grid = (splits, nh, B); the `splits` CTAs of one (sequence, head) form a thread-block cluster and share the keys.
//   1  scores: DH / 16 adjacent lanes cover one key (16 bytes each, dp4a against the query slice held in registers,
//      shuffle reduction); a thread keeps four keys in flight.  t = d~ log2(e) (q . k) goes to shared memory.
//   2  CTA maximum m_c, e = 2^(t - m_c) in place, CTA sum l_c; (m_c, l_c) are exchanged through distributed shared
//      memory: m = max m_c, l = sum l_c 2^(m_c - m) in rank order.
//   3  P_u8 = clip(Round(e 2^(m_c - m) / (l s_p)))  (row-max mode: Round(255 e 2^(m_c - m))), one byte per key.
//   4  acc[d] = sum_k P_u8[k] V[k][d]: same lane layout as step 1; the four keys a thread holds are transposed with
//      byte permutes so that one dp4a applies four keys' probabilities to one feature; a quad whose four
//      probabilities are all zero is not fetched.  INT32 partial sums: exact in any order.
//   5  the partial sums are added across key groups (shared memory) and across the cluster (distributed shared
//      memory); rank 0 applies s_p s_v and the output stage (FWQ / SQ INT8, or F16 / BF16).
// The new token's key / value may come from a separate buffer (the QKV GeMM^quant output); rank 0 then also stores
// them into the cache, so that no separate append kernel runs.
#include "common.cuh"
#include "ptx.cuh"
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

constexpr int DEC_MAX_CHUNK = 12288;          // keys per CTA: 4 bytes of score + 1 byte of P each, within 64 KB
constexpr int DEC_MAX_SPLITS = 8;             // portable cluster size
constexpr float DEC_MAGIC = 12582912.0f;      // 1.5 * 2^23

struct DecodeParams {
  const int8_t* q; long long ld_q;
  int8_t* kc; int8_t* vc; long long ld_kv, bstride;
  const int8_t* k_new; const int8_t* v_new; long long ld_new;
  const int* len;
  int max_len;              // the launch is sized for this many keys: a larger len[b] is clamped to it
  int nh;
  float score_scale;        // d~ log2(e)
  float pv_scale;           // static: s_p s_v; row-max: s_v / 255
  float inv_sp;             // 1 / s_p
  int rowmax;
  const float* out_scale; int out_scale_stride;   // FWQ [H] (stride 1) / SQ [1] (stride 0); NULL for an FP output
  void* out; long long out_ld; int out_dt;
  int chunk_cap;            // score slots in shared memory (multiple of 16)
};

__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {      // signed x signed bytes
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ int dp4a_su(uint32_t a, uint32_t b, int c) {      // signed bytes of a x unsigned bytes of b
  int d;
  asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t dec_ld_cluster(uint32_t cluster_addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// NT threads per CTA: 128 when the launch has CTAs to spare, 256 when (sequence, head) pairs are few and every CTA has
// to keep more loads in flight.
template <int DH, int NT>
__global__ void __launch_bounds__(NT) attn_decode_kernel(const DecodeParams p) {
  constexpr int U = 1;                         // key quads in flight per thread (two measured slower: 37 against 27 us on B8 S2048 dh128)
  constexpr int DEC_THREADS = NT, DEC_WARPS = NT / 32;
  constexpr int TPK = DH / 16;                 // lanes per key
  constexpr int G = DEC_THREADS / TPK;         // key quads per CTA sweep
  extern __shared__ __align__(16) uint8_t dsm[];
  float* sc = reinterpret_cast<float*>(dsm);                        // [chunk_cap] scores, then exponentials
  uint32_t* pw = reinterpret_cast<uint32_t*>(sc + p.chunk_cap);     // [chunk_cap / 4] four P_u8 per word
  int* red = reinterpret_cast<int*>(pw + p.chunk_cap / 4);          // [warps][DH] partial sums of the warps
  int* part = red + DEC_WARPS * DH;                                         // [DH] this CTA's partial sums
  float* xch = reinterpret_cast<float*>(part + DH);                 // [2] (m_c, l_c)
  float* wred = xch + 2;                                            // [DEC_WARPS] per-warp scratch

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = tid % TPK, g = tid / TPK;
  const int splits = gridDim.x, rank = (int)ptx::cluster_ctarank();
  const int h = blockIdx.y, b = blockIdx.z;
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();
  const int L = min(__ldg(p.len + b), p.max_len);
  const int col = h * DH + c * 16;

  if (L <= 0) {                                                     // uniform over the cluster: nobody reaches a barrier
    if (rank == 0 && tid < DH) {
      const long long at = (long long)b * p.out_ld + h * DH + tid;
      if (p.out_dt == HERO_I8) reinterpret_cast<int8_t*>(p.out)[at] = 0;
      else reinterpret_cast<uint16_t*>(p.out)[at] = 0;
    }
    return;
  }
  // this CTA's keys [k0, k1): equal shares, multiples of 4
  const int per = (((L + splits - 1) / splits) + 3) & ~3;
  const int k0 = min(rank * per, L), k1 = min(k0 + per, L), n = k1 - k0;
  const int nq = (n + 3) >> 2;
  const int8_t* kbase = p.kc + (long long)b * p.bstride + col;
  const int8_t* vbase = p.vc + (long long)b * p.bstride + col;
  const bool fresh = p.k_new != nullptr;                            // entry L - 1 comes from k_new / v_new
  auto krow = [&](int k) -> const uint4* {
    return reinterpret_cast<const uint4*>((fresh && k == L - 1) ? p.k_new + (long long)b * p.ld_new + col : kbase + (long long)k * p.ld_kv);
  };
  auto vrow = [&](int k) -> const uint4* {
    return reinterpret_cast<const uint4*>((fresh && k == L - 1) ? p.v_new + (long long)b * p.ld_new + col : vbase + (long long)k * p.ld_kv);
  };

  // ---- 1: scores
  const uint4 qv = __ldg(reinterpret_cast<const uint4*>(p.q + (long long)b * p.ld_q + col));
  float mloc = -INFINITY;
  for (int q0 = 0; q0 < nq; q0 += U * G) {                  // trip count uniform over the warp: the shuffles below need every lane
    uint4 kv[U][4];                                          // U quads = 4 U keys in flight per thread
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j < 4; ++j) kv[u][j] = __ldg(krow(min(k0 + 4 * (q0 + u * G + g) + j, k1 - 1)));
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int qd = q0 + u * G + g;
      float t[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int a = dp4a_ss(kv[u][j].x, qv.x, 0);
        a = dp4a_ss(kv[u][j].y, qv.y, a);
        a = dp4a_ss(kv[u][j].z, qv.z, a);
        a = dp4a_ss(kv[u][j].w, qv.w, a);
#pragma unroll
        for (int o = 1; o < TPK; o <<= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        t[j] = (4 * qd + j < n) ? (float)a * p.score_scale : -INFINITY;
        mloc = fmaxf(mloc, t[j]);
      }
      if (c == 0 && qd < nq) *reinterpret_cast<float4*>(sc + 4 * qd) = make_float4(t[0], t[1], t[2], t[3]);
    }
  }
  // rank 0 appends the new token to the cache (its own lanes cover the row once)
  if (fresh && rank == 0 && g == 0) {
    *reinterpret_cast<uint4*>(p.kc + (long long)b * p.bstride + (long long)(L - 1) * p.ld_kv + col) = __ldg(krow(L - 1));
    *reinterpret_cast<uint4*>(p.vc + (long long)b * p.bstride + (long long)(L - 1) * p.ld_kv + col) = __ldg(vrow(L - 1));
  }
  mloc = warp_max(mloc);
  if (lane == 0) wred[warp] = mloc;
  __syncthreads();
  float m_c = wred[0];                                       // -inf when this CTA has no key
#pragma unroll
  for (int w = 1; w < DEC_WARPS; ++w) m_c = fmaxf(m_c, wred[w]);
  __syncthreads();

  // ---- 2: exponentials in place, CTA sum
  float lloc = 0.f;
  for (int k = tid; k < 4 * nq; k += DEC_THREADS) {
    const float e = (k < n) ? exp2f(sc[k] - m_c) : 0.f;
    sc[k] = e;
    lloc += e;
  }
  lloc = warp_sum(lloc);
  if (lane == 0) wred[warp] = lloc;
  __syncthreads();
  if (tid == 0) {
    float lc = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) lc += wred[w];
    xch[0] = m_c; xch[1] = lc;
  }
  ptx::cluster_sync();
  float m = -INFINITY, l = 0.f;
  {
    const uint32_t xa = ptx::smem_u32(xch);
    float mq[DEC_MAX_SPLITS], lq[DEC_MAX_SPLITS];
#pragma unroll
    for (int q = 0; q < DEC_MAX_SPLITS; ++q) {
      mq[q] = q < splits ? __uint_as_float(dec_ld_cluster(ptx::mapa(xa, q))) : -INFINITY;
      lq[q] = q < splits ? __uint_as_float(dec_ld_cluster(ptx::mapa(xa + 4, q))) : 0.f;
      m = fmaxf(m, mq[q]);
    }
#pragma unroll
    for (int q = 0; q < DEC_MAX_SPLITS; ++q) l += (mq[q] == -INFINITY) ? 0.f : lq[q] * exp2f(mq[q] - m);
  }

  // ---- 3: P_u8, four keys per word
  {
    const float f = (n > 0 ? exp2f(m_c - m) : 0.f) * (p.rowmax ? 255.0f : p.inv_sp / l);
    for (int qd = tid; qd < nq; qd += DEC_THREADS) {
      const float4 e = *reinterpret_cast<const float4*>(sc + 4 * qd);
      const float a0 = fminf(e.x * f, 255.0f) + DEC_MAGIC, a1 = fminf(e.y * f, 255.0f) + DEC_MAGIC;
      const float a2 = fminf(e.z * f, 255.0f) + DEC_MAGIC, a3 = fminf(e.w * f, 255.0f) + DEC_MAGIC;
      const uint32_t lo = __byte_perm(__float_as_uint(a0), __float_as_uint(a1), 0x0040);
      const uint32_t hi = __byte_perm(__float_as_uint(a2), __float_as_uint(a3), 0x0040);
      pw[qd] = __byte_perm(lo, hi, 0x5410);
    }
  }
  __syncthreads();

  // ---- 4: acc[d] += P_u8[k] V[k][d]
  int acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0;
  for (int q0 = g; q0 < nq; q0 += U * G) {
    uint32_t p4[U], any = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) { p4[u] = (q0 + u * G < nq) ? pw[q0 + u * G] : 0u; any |= p4[u]; }
    if (any == 0) continue;
    uint4 vv[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (p4[u] != 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) vv[u][j] = __ldg(vrow(min(k0 + 4 * (q0 + u * G) + j, k1 - 1)));
      }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (p4[u] == 0) continue;
      const uint32_t x[4][4] = {{vv[u][0].x, vv[u][1].x, vv[u][2].x, vv[u][3].x}, {vv[u][0].y, vv[u][1].y, vv[u][2].y, vv[u][3].y},
                                {vv[u][0].z, vv[u][1].z, vv[u][2].z, vv[u][3].z}, {vv[u][0].w, vv[u][1].w, vv[u][2].w, vv[u][3].w}};
#pragma unroll
      for (int w = 0; w < 4; ++w) {                            // features 4 w .. 4 w + 3 of this lane's slice
        const uint32_t ab = __byte_perm(x[w][0], x[w][1], 0x5140), cd = __byte_perm(x[w][2], x[w][3], 0x5140);
        const uint32_t ef = __byte_perm(x[w][0], x[w][1], 0x7362), gh = __byte_perm(x[w][2], x[w][3], 0x7362);
        acc[4 * w + 0] = dp4a_su(__byte_perm(ab, cd, 0x5410), p4[u], acc[4 * w + 0]);
        acc[4 * w + 1] = dp4a_su(__byte_perm(ab, cd, 0x7632), p4[u], acc[4 * w + 1]);
        acc[4 * w + 2] = dp4a_su(__byte_perm(ef, gh, 0x5410), p4[u], acc[4 * w + 2]);
        acc[4 * w + 3] = dp4a_su(__byte_perm(ef, gh, 0x7632), p4[u], acc[4 * w + 3]);
      }
    }
  }
  // ---- 5: key groups of a warp (shuffles) -> warps (shared memory) -> cluster -> output stage
#pragma unroll
  for (int i = 0; i < 16; ++i)
#pragma unroll
    for (int o = TPK; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
  if (lane < TPK) {
#pragma unroll
    for (int i = 0; i < 16; i += 4)
      *reinterpret_cast<int4*>(red + warp * DH + c * 16 + i) = make_int4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
  }
  __syncthreads();
  if (tid < DH) {
    int s = 0;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) s += red[w * DH + tid];
    part[tid] = s;
  }
  ptx::cluster_sync();
  if (rank == 0 && tid < DH) {
    const uint32_t pa = ptx::smem_u32(part + tid);
    int s = 0;
#pragma unroll
    for (int q = 0; q < DEC_MAX_SPLITS; ++q) s += q < splits ? (int)dec_ld_cluster(ptx::mapa(pa, q)) : 0;
    const int d = h * DH + tid;
    const long long at = (long long)b * p.out_ld + d;
    const float rowf = p.rowmax ? 1.0f / l : 1.0f;
    if (p.out_dt == HERO_I8) {
      const float fac = p.pv_scale / __ldg(p.out_scale + (long long)d * p.out_scale_stride);
      const float r = fminf(fmaxf((float)s * rowf * fac, -127.f), 127.f) + DEC_MAGIC;
      reinterpret_cast<int8_t*>(p.out)[at] = (int8_t)(__float_as_uint(r) & 0xff);
    } else {
      const float x = (float)s * rowf * p.pv_scale;
      if (p.out_dt == HERO_F16) reinterpret_cast<__half*>(p.out)[at] = __float2half_rn(x);
      else reinterpret_cast<__nv_bfloat16*>(p.out)[at] = __float2bfloat16_rn(x);
    }
  }
  ptx::cluster_sync();                                       // nobody leaves while rank 0 may still read its sums
}

template <int DH, int NT>
static hero_status launch_decode(hero_handle* h, const DecodeParams& p, int B, int splits, cudaStream_t stream) {
  auto kern = attn_decode_kernel<DH, NT>;
  const size_t smem = (size_t)p.chunk_cap * 5 + (size_t)(NT / 32 * DH + DH) * 4 + 8 + NT / 32 * 4 + 16;
  static PerDeviceInt configured;    // largest opt-in made so far, per device
  if (smem > 48 * 1024 && (int)smem > configured.get(h->device)) {
    HERO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured.set(h->device, (int)smem);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)splits, (unsigned)p.nh, (unsigned)B);
  cfg.blockDim = dim3(NT);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)splits; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_take_fence(stream) ? 1 : 2;   // a fenced stream: ordinary serialisation
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    HERO_CUDA(cudaLaunchKernelEx(&cfg, kern, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero

extern "C" hero_status hero_int8_decode_attention(hero_handle* h, const hero_decode_attn_args* a, void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && a, HERO_ERR_INVALID_ARG, "hero_int8_decode_attention: NULL handle or args");
  HERO_REQUIRE(a->q && a->k_cache && a->v_cache && a->len, HERO_ERR_INVALID_ARG, "q, k_cache, v_cache and len are required");
  HERO_REQUIRE(a->B >= 0 && a->nh > 0 && (a->dh == 64 || a->dh == 128), HERO_ERR_UNSUPPORTED, "B=%d nh=%d dh=%d: dh must be 64 or 128",
               a->B, a->nh, a->dh);
  const long long H = (long long)a->nh * a->dh;
  HERO_REQUIRE(a->max_len >= 1 && a->max_len <= DEC_MAX_SPLITS * DEC_MAX_CHUNK, HERO_ERR_UNSUPPORTED, "max_len=%d: 1 .. %d supported",
               a->max_len, DEC_MAX_SPLITS * DEC_MAX_CHUNK);
  HERO_REQUIRE((a->k_new == nullptr) == (a->v_new == nullptr), HERO_ERR_INVALID_ARG, "k_new and v_new go together");
  HERO_REQUIRE(aligned16(a->q) && aligned16(a->k_cache) && aligned16(a->v_cache) && aligned16(a->k_new) && aligned16(a->v_new),
               HERO_ERR_ALIGNMENT, "q, caches and new rows must be 16-byte aligned");
  HERO_REQUIRE(a->ld_q >= H && a->ld_q % 16 == 0 && a->ld_kv >= H && a->ld_kv % 16 == 0 && a->batch_stride % 16 == 0 &&
               a->batch_stride >= (long long)a->max_len * a->ld_kv, HERO_ERR_ALIGNMENT,
               "ld_q, ld_kv >= nh*dh, batch_stride >= max_len * ld_kv, all multiples of 16");
  if (a->k_new) HERO_REQUIRE(a->ld_new >= H && a->ld_new % 16 == 0, HERO_ERR_ALIGNMENT, "ld_new >= nh*dh and a multiple of 16");
  HERO_REQUIRE(a->p_mode == HERO_P_STATIC || a->p_mode == HERO_P_ROWMAX, HERO_ERR_INVALID_ARG, "p_mode %d", a->p_mode);
  HERO_REQUIRE(a->s_q > 0.f && a->s_k > 0.f && a->s_v > 0.f && (a->p_mode == HERO_P_ROWMAX || a->s_p > 0.f), HERO_ERR_INVALID_ARG,
               "s_q, s_k, s_v, s_p must be positive");
  hero_status st;
  if ((st = check_matrix(a->out, "out")) != HERO_OK) return st;
  HERO_REQUIRE(a->out.rows == a->B && a->out.cols == H, HERO_ERR_INVALID_ARG, "out must be [B, nh*dh]");
  HERO_REQUIRE(a->out.dtype == HERO_I8 || is_fp16ish(a->out.dtype), HERO_ERR_UNSUPPORTED, "out dtype %d: INT8, F16 or BF16", a->out.dtype);
  if (a->out.dtype == HERO_I8)
    HERO_REQUIRE((a->out.gran == HERO_GRAN_FWQ || a->out.gran == HERO_GRAN_SQ) && a->out.scale, HERO_ERR_INVALID_ARG,
                 "an INT8 X_attn carries a feature-wise or static scale");
  if (a->B == 0) return HERO_OK;

  DecodeParams p;
  memset(&p, 0, sizeof(p));
  p.q = static_cast<const int8_t*>(a->q); p.ld_q = a->ld_q;
  p.kc = static_cast<int8_t*>(a->k_cache); p.vc = static_cast<int8_t*>(a->v_cache); p.ld_kv = a->ld_kv; p.bstride = a->batch_stride;
  p.k_new = static_cast<const int8_t*>(a->k_new); p.v_new = static_cast<const int8_t*>(a->v_new); p.ld_new = a->ld_new;
  p.len = a->len; p.max_len = a->max_len; p.nh = a->nh;
  p.score_scale = a->s_q * a->s_k / sqrtf((float)a->dh) * 1.4426950408889634f;
  p.rowmax = a->p_mode == HERO_P_ROWMAX;
  p.pv_scale = p.rowmax ? a->s_v / 255.0f : a->s_p * a->s_v;
  p.inv_sp = p.rowmax ? 0.f : 1.0f / a->s_p;
  p.out_scale = a->out.dtype == HERO_I8 ? a->out.scale : nullptr;
  p.out_scale_stride = a->out.gran == HERO_GRAN_FWQ ? 1 : 0;
  p.out = a->out.data; p.out_ld = a->out.ld; p.out_dt = a->out.dtype;
  // key splits: enough CTAs for about four per SM, at least 512 keys each, as many as the score buffer requires
  int splits = 1;
  const long long heads = (long long)a->B * a->nh;
  while (splits < DEC_MAX_SPLITS && (heads * splits < 4ll * h->sm_count && a->max_len / (splits * 2) >= 512)) splits *= 2;
  while (splits < DEC_MAX_SPLITS && (a->max_len + splits - 1) / splits > DEC_MAX_CHUNK) splits *= 2;
  p.chunk_cap = (((a->max_len + splits - 1) / splits) + 4 + 15) & ~15;   // multiple of 16: the arrays behind it stay 16-byte aligned
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // few (sequence, head) pairs: wider CTAs keep more loads in flight per SM (38 against 59 us on B1 S16384 dh128)
  if (heads * splits <= 2ll * h->sm_count)
    return a->dh == 64 ? launch_decode<64, 256>(h, p, a->B, splits, s) : launch_decode<128, 256>(h, p, a->B, splits, s);
  return a->dh == 64 ? launch_decode<64, 128>(h, p, a->B, splits, s) : launch_decode<128, 128>(h, p, a->B, splits, s);
}
