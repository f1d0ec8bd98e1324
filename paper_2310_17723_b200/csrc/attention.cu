// INT8 attention core (Sec. 2.2.2 Eq. 15-17): A = d~ Q K^T (INT32 -> fp32, never quantized),
// P = softmax(A), P_u8 = Round(P / s_p) requantized ON CHIP to unsigned 8 bit, acc = P_u8 V (INT32),
// X_attn = Round(acc * s_p s_v / S_attn[j]).
//
// The static scalar s_p quantizes the FULLY NORMALISED probability, so the final row max and row sum
// must be known before any P is rounded: the kernel makes two sweeps over the keys.  Sweep 1 runs
// Q K^T per 128-key block on the tensor cores and keeps only running (max, sum) per row; sweep 2
// recomputes each block's scores, turns them into P_u8, stores them in shared memory in the UMMA
// operand layout and accumulates P_u8 V in tensor memory.  INT8 Q K^T is cheap enough (one eighth of
// the exponential cost) that recomputing beats spilling the scores.
//
// One CTA per (batch, head, 128-query tile); 10 warps:
//   warps 0-7  softmax / epilogue: row r = 32 * (w % 4) + lane, columns 64 * (w / 4) .. +63 of a block
//   warp  8    TMA producer (Q once, K per block and sweep, V per block in sweep 2)
//   warp  9    UMMA issuer (one lane) and owner of the TMEM allocation
// TMEM: two score buffers of 128 columns (double-buffered against the softmax warps) + dh output columns.
#include "common.cuh"
#include "ptx.cuh"
#include <climits>
#include <cmath>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

constexpr int ATT_BM = 128;      // queries per CTA
constexpr int ATT_BN = 128;      // keys per block
constexpr int ATT_THREADS = 320;
constexpr int ATT_KSTAGES = 3;
constexpr int ATT_VSTAGES = 2;

struct AttnParams {
  int B, S, nh, dh;
  int nqt;                 // query tiles per sequence
  float c2;                // d~ * log2(e),  d~ = s_q s_k / sqrt(dh)
  float inv_sp;            // 1 / s_p
  float pv_scale;          // s_p * s_v
  const float* out_scale;  // FWQ [H] (stride 1) / SQ [1] (stride 0); NULL for an FP output
  int out_scale_stride;
  int mask;
  const int* key_len;
  void* out;
  long long out_ld;
  int out_dt;
  uint32_t idesc_qk, idesc_pv;
  int* err;
};

template <int DH>
struct AttnCfg {
  static constexpr int TILE = ATT_BM * DH;                     // bytes of a Q / K / V tile (INT8)
  static constexpr int P_TILE = ATT_BM * ATT_BN;               // bytes of a P_u8 tile
  static constexpr int OFF_K = TILE;
  static constexpr int OFF_V = OFF_K + ATT_KSTAGES * TILE;
  static constexpr int OFF_P = OFF_V + ATT_VSTAGES * TILE;
  static constexpr int OFF_STATS = OFF_P + 2 * P_TILE;         // float2 [2][128]
  static constexpr int OFF_BARS = OFF_STATS + 2 * ATT_BM * 8;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + 32 * 8 + 16;
  static constexpr uint32_t SWZ = (DH == 128) ? ptx::SWZ_128B : ptx::SWZ_64B;
  static constexpr uint32_t SBO = 8 * DH;                      // 8 rows of DH bytes
  static constexpr int TMEM_COLS = 512;
  static constexpr int O_COL = 256;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t sat_u8(float x) {
  uint32_t r;
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void st_shared16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_g16(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t q4(float a, float b, float c, float d) {
  int ia = __float2int_rn(fminf(fmaxf(a, -127.f), 127.f));
  int ib = __float2int_rn(fminf(fmaxf(b, -127.f), 127.f));
  int ic = __float2int_rn(fminf(fmaxf(c, -127.f), 127.f));
  int id = __float2int_rn(fminf(fmaxf(d, -127.f), 127.f));
  return (uint32_t)(ia & 0xff) | ((uint32_t)(ib & 0xff) << 8) | ((uint32_t)(ic & 0xff) << 16) | ((uint32_t)id << 24);
}
__device__ __forceinline__ uint32_t fp2(float a, float b, int dt) {
  if (dt == HERO_F16) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_int8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using Cfg = AttnCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + Cfg::OFF_K;
  uint8_t* sV = smem + Cfg::OFF_V;
  uint8_t* sP = smem + Cfg::OFF_P;
  float2* stats = reinterpret_cast<float2*>(smem + Cfg::OFF_STATS);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BARS);
  uint64_t* q_full = bars;            // 1
  uint64_t* k_full = bars + 1;        // 3
  uint64_t* k_empty = bars + 4;       // 3
  uint64_t* v_full = bars + 7;        // 2
  uint64_t* v_empty = bars + 9;       // 2
  uint64_t* s_full = bars + 11;       // 2
  uint64_t* s_empty = bars + 13;      // 2   (8 arrivals: one per softmax warp)
  uint64_t* p_full = bars + 15;       // 2   (8 arrivals)
  uint64_t* p_empty = bars + 17;      // 2
  uint64_t* o_full = bars + 19;       // 1
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- which tile: heavy (late) query tiles first so that causal work balances
  int idx = blockIdx.x;
  const int qt = p.nqt - 1 - (idx % p.nqt); idx /= p.nqt;
  const int h = idx % p.nh;
  const int b = idx / p.nh;
  const int q0 = qt * ATT_BM;
  int klen = p.S;
  if (p.key_len) klen = min(p.S, max(0, p.key_len[b]));
  int kv_end = klen;
  if (p.mask == HERO_MASK_CAUSAL) kv_end = min(kv_end, q0 + ATT_BM);
  const int nkv = (kv_end + ATT_BN - 1) / ATT_BN;
  const int row_base = b * p.S;           // first row of this sequence in the [B*S, .] views
  const int col0 = h * DH;

  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    for (int i = 0; i < ATT_KSTAGES; ++i) { ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < ATT_VSTAGES; ++i) { ptx::mbar_init(&v_full[i], 1); ptx::mbar_init(&v_empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_empty[i], 8);
      ptx::mbar_init(&p_full[i], 8); ptx::mbar_init(&p_empty[i], 1);
    }
    ptx::mbar_init(o_full, 1);
    ptx::fence_mbar_init();
  }
  if (warp == 9) { ptx::tmem_alloc(tmem_slot, Cfg::TMEM_COLS); ptx::tmem_relinquish(); }
  if (warp == 8 && lane == 0) { ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && nkv > 0) {
      ptx::mbar_expect_tx(q_full, Cfg::TILE);
      ptx::tma_load_2d(sQ, &tmQ, col0, row_base + q0, q_full);
      bool ok = true;
      for (int i = 0; i < 2 * nkv && ok; ++i) {
        const int j = i < nkv ? i : i - nkv;
        const int ks = i % ATT_KSTAGES;
        const uint32_t kph = (i / ATT_KSTAGES) & 1;
        if (!ptx::mbar_wait(&k_empty[ks], kph ^ 1, p.err, 0x1100 | ks)) { ok = false; break; }
        ptx::mbar_expect_tx(&k_full[ks], Cfg::TILE);
        ptx::tma_load_2d(sK + ks * Cfg::TILE, &tmK, col0, row_base + j * ATT_BN, &k_full[ks]);
        if (i >= nkv) {
          const int vs = j % ATT_VSTAGES;
          const uint32_t vph = (j / ATT_VSTAGES) & 1;
          if (!ptx::mbar_wait(&v_empty[vs], vph ^ 1, p.err, 0x1200 | vs)) { ok = false; break; }
          ptx::mbar_expect_tx(&v_full[vs], Cfg::TILE);
          ptx::tma_load_2d(sV + vs * Cfg::TILE, &tmV, col0, row_base + j * ATT_BN, &v_full[vs]);
        }
      }
      // drain: the last copies have landed (and been consumed) before the CTA may exit
      if (ok) ptx::mbar_wait(o_full, 0, p.err, 0x1300);
    }
    __syncwarp();
  } else if (warp == 9) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0 && nkv > 0) {
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // Q, K: K-major rows of DH bytes
      constexpr uint64_t pmaj = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);      // P: K-major rows of 128 bytes
      constexpr uint64_t vmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // V: MN-major, 8-key groups
      bool ok = ptx::mbar_wait(q_full, 0, p.err, 0x2000);
      const uint32_t q_addr = ptx::smem_u32(sQ);

      auto issue_pv = [&](int j) -> bool {
        const int vs = j % ATT_VSTAGES, pb = j & 1;
        if (!ptx::mbar_wait(&v_full[vs], (j / ATT_VSTAGES) & 1, p.err, 0x2100 | vs)) return false;
        if (!ptx::mbar_wait(&p_full[pb], (j >> 1) & 1, p.err, 0x2200 | pb)) return false;
        ptx::tc_fence_after();
        const uint32_t p_addr = ptx::smem_u32(sP + pb * Cfg::P_TILE);
        const uint32_t v_addr = ptx::smem_u32(sV + vs * Cfg::TILE);
#pragma unroll
        for (int k = 0; k < ATT_BN / 32; ++k)
          ptx::umma_i8(tmem_base + Cfg::O_COL, ptx::smem_desc(pmaj, p_addr + k * 32),
                       ptx::smem_desc(vmaj, v_addr + k * 32 * DH), p.idesc_pv, (j | k) != 0);
        ptx::umma_commit(&v_empty[vs]);
        ptx::umma_commit(&p_empty[pb]);
        return true;
      };

      for (int i = 0; i < 2 * nkv && ok; ++i) {
        const int ks = i % ATT_KSTAGES, sb = i & 1;
        if (!ptx::mbar_wait(&k_full[ks], (i / ATT_KSTAGES) & 1, p.err, 0x2300 | ks)) { ok = false; break; }
        if (!ptx::mbar_wait(&s_empty[sb], ((i >> 1) & 1) ^ 1, p.err, 0x2400 | sb)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t k_addr = ptx::smem_u32(sK + ks * Cfg::TILE);
#pragma unroll
        for (int k = 0; k < DH / 32; ++k)
          ptx::umma_i8(tmem_base + sb * ATT_BN, ptx::smem_desc(kmaj, q_addr + k * 32),
                       ptx::smem_desc(kmaj, k_addr + k * 32), p.idesc_qk, k != 0);
        ptx::umma_commit(&k_empty[ks]);
        ptx::umma_commit(&s_full[sb]);
        if (i >= nkv + 1) ok = issue_pv(i - nkv - 1);
      }
      if (ok) ok = issue_pv(nkv - 1);
      if (ok) ptx::umma_commit(o_full);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    const int quarter = warp & 3, half = warp >> 2;
    const int r_loc = quarter * 32 + lane;
    const int q = q0 + r_loc;
    const bool row_ok = q < p.S;
    int kmax = klen - 1;                                     // last allowed key (inclusive)
    if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;
    bool ok = true;

    float m = -INFINITY, l = 0.f;
    // ---- sweep 1: running row max and row sum (log2 domain)
    for (int i = 0; i < nkv; ++i) {
      const int sb = i & 1;
      if (ok && !ptx::mbar_wait(&s_full[sb], (i >> 1) & 1, p.err, 0x3000 | sb)) ok = false;
      ptx::tc_fence_after();
      if (ok) {
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + half * 64 + cc * 32, r);
          ptx::tmem_ld_wait();
          const int kb = i * ATT_BN + half * 64 + cc * 32;
          const int nvalid = min(32, kmax - kb + 1);       // keys kb .. kb + nvalid - 1 are allowed
          if (nvalid <= 0) continue;
          int imax = INT_MIN;
          if (nvalid == 32) {
#pragma unroll
            for (int j = 0; j < 32; ++j) imax = max(imax, (int)r[j]);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) imax = max(imax, j < nvalid ? (int)r[j] : INT_MIN);
          }
          const float m_new = fmaxf(m, (float)imax * c2);
          float acc = 0.f;
          if (nvalid == 32) {
#pragma unroll
            for (int j = 0; j < 32; ++j) acc += ex2f(fmaf((float)(int)r[j], c2, -m_new));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) acc += j < nvalid ? ex2f(fmaf((float)(int)r[j], c2, -m_new)) : 0.f;
          }
          l = l * ex2f(m - m_new) + acc;                    // m = -inf on first use: 2^-inf = 0
          m = m_new;
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&s_empty[sb]);
    }
    // ---- combine the two column halves of each row
    stats[half * ATT_BM + r_loc] = make_float2(m, l);
    asm volatile("bar.sync 1, 256;" ::: "memory");
    {
      const float2 o = stats[(half ^ 1) * ATT_BM + r_loc];
      const float mf = fmaxf(m, o.x);
      float lf = 0.f;
      if (mf > -INFINITY) lf = (m > -INFINITY ? l * ex2f(m - mf) : 0.f) + (o.x > -INFINITY ? o.y * ex2f(o.x - mf) : 0.f);
      m = mf; l = lf;
    }
    // P_u8 = Round(P / s_p) with P = 2^(t - m) / l
    const float pscale = l > 0.f ? p.inv_sp / l : 0.f;

    // ---- sweep 2: scores again -> P_u8 in shared memory (UMMA K-major, 128-byte swizzle)
    for (int j = 0; j < nkv; ++j) {
      const int i = nkv + j, sb = i & 1, pb = j & 1;
      if (ok && !ptx::mbar_wait(&s_full[sb], (i >> 1) & 1, p.err, 0x3100 | sb)) ok = false;
      if (ok && !ptx::mbar_wait(&p_empty[pb], ((j >> 1) & 1) ^ 1, p.err, 0x3200 | pb)) ok = false;
      ptx::tc_fence_after();
      if (ok) {
        const uint32_t prow = ptx::smem_u32(sP + pb * Cfg::P_TILE) + (r_loc >> 3) * 1024 + (r_loc & 7) * 128;
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + half * 64 + cc * 32, r);
          ptx::tmem_ld_wait();
          const int kb = j * ATT_BN + half * 64 + cc * 32;
          const int nvalid = min(32, kmax - kb + 1);
          uint32_t w[8];
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            uint32_t word = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int jj = 4 * g + e;
              float pe = ex2f(fmaf((float)(int)r[jj], c2, -m)) * pscale;
              if (jj >= nvalid) pe = 0.f;
              word |= sat_u8(pe) << (8 * e);
            }
            w[g] = word;
          }
          const int c16 = half * 4 + cc * 2;                // 16-byte chunk index within the 128-byte row
          st_shared16(prow + (((c16) ^ (r_loc & 7)) << 4), w[0], w[1], w[2], w[3]);
          st_shared16(prow + (((c16 + 1) ^ (r_loc & 7)) << 4), w[4], w[5], w[6], w[7]);
        }
      }
      ptx::tc_fence_before();
      ptx::fence_proxy_async_smem();                         // generic-proxy writes -> visible to the UMMA (async proxy)
      __syncwarp();
      if (lane == 0) { ptx::mbar_arrive(&s_empty[sb]); ptx::mbar_arrive(&p_full[pb]); }
    }

    // ---- epilogue: X_attn = acc * s_p s_v (/ S_attn[j] -> Round -> INT8)
    if (nkv > 0 && ok && !ptx::mbar_wait(o_full, 0, p.err, 0x3300)) ok = false;
    ptx::tc_fence_after();
    constexpr int NCH = DH / 64;                             // 32-column chunks per half
#pragma unroll 1
    for (int cc = 0; cc < NCH; ++cc) {
      uint32_t r[32];
      const int ocol = half * (DH / 2) + cc * 32;
      if (nkv > 0 && ok) {
        ptx::tmem_ld32(t_lane + Cfg::O_COL + ocol, r);
        ptx::tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = 0;               // every key masked: the row is zero
      }
      if (!row_ok) continue;
      const long long grow = (long long)(row_base + q);
      const int gcol = col0 + ocol;
      if (p.out_dt == HERO_I8) {
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j)
          v[j] = (float)(int)r[j] * (p.pv_scale / __ldg(p.out_scale + (gcol + j) * p.out_scale_stride));
        int8_t* dst = reinterpret_cast<int8_t*>(p.out) + grow * p.out_ld + gcol;
#pragma unroll
        for (int g = 0; g < 2; ++g)
          st_g16(dst + 16 * g, q4(v[16 * g], v[16 * g + 1], v[16 * g + 2], v[16 * g + 3]),
                 q4(v[16 * g + 4], v[16 * g + 5], v[16 * g + 6], v[16 * g + 7]),
                 q4(v[16 * g + 8], v[16 * g + 9], v[16 * g + 10], v[16 * g + 11]),
                 q4(v[16 * g + 12], v[16 * g + 13], v[16 * g + 14], v[16 * g + 15]));
      } else {
        uint16_t* dst = reinterpret_cast<uint16_t*>(p.out) + grow * p.out_ld + gcol;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float v[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) v[e] = (float)(int)r[8 * g + e] * p.pv_scale;
          st_g16(dst + 8 * g, fp2(v[0], v[1], p.out_dt), fp2(v[2], v[3], p.out_dt), fp2(v[4], v[5], p.out_dt),
                 fp2(v[6], v[7], p.out_dt));
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 9) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int DH>
static hero_status launch_attn(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = AttnCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  CUtensorMap tq, tk, tv;
  hero_status st;
  if ((st = make_tmap_2d(h, &tq, a->q, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BM, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  p.idesc_qk = ptx::make_idesc(2, 1, 1, 0, 0, ATT_BM, ATT_BN);   // S8 x S8 -> S32, both K-major
  p.idesc_pv = ptx::make_idesc(2, 0, 1, 0, 1, ATT_BM, DH);       // U8 x S8 -> S32, V is MN-major
  auto kern = attn_int8_kernel<DH>;
  static bool configured = false;
  if (!configured) {
    HERO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES));
    configured = true;
  }
  const long long grid = (long long)p.nqt * a->nh * a->B;
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    kern<<<(unsigned)grid, ATT_THREADS, Cfg::SMEM_BYTES, stream>>>(tq, tk, tv, p);
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero

extern "C" hero_status hero_int8_attention(hero_handle* h, const hero_attn_args* a, void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && a, HERO_ERR_INVALID_ARG, "hero_int8_attention: NULL handle or args");
  HERO_REQUIRE(a->q && a->k && a->v, HERO_ERR_INVALID_ARG, "q, k, v are required");
  HERO_REQUIRE(a->B >= 0 && a->S > 0 && a->nh > 0, HERO_ERR_INVALID_ARG, "bad B / S / nh");
  HERO_REQUIRE(a->dh == 64 || a->dh == 128, HERO_ERR_UNSUPPORTED, "dh=%d: 64 or 128 supported", a->dh);
  HERO_REQUIRE(a->dtype == HERO_I8, HERO_ERR_UNSUPPORTED, "q/k/v dtype %d: this build runs the INT8 core only", a->dtype);
  HERO_REQUIRE(aligned16(a->q) && aligned16(a->k) && aligned16(a->v) && a->ld % 16 == 0 && a->ld >= (int64_t)a->nh * a->dh,
               HERO_ERR_ALIGNMENT, "q/k/v must be 16-byte aligned with ld a multiple of 16 and >= nh*dh");
  hero_status st;
  if ((st = check_matrix(a->out, "out")) != HERO_OK) return st;
  HERO_REQUIRE(a->out.rows == (int64_t)a->B * a->S && a->out.cols == (int64_t)a->nh * a->dh, HERO_ERR_INVALID_ARG,
               "out must be [B*S, nh*dh]");
  HERO_REQUIRE(a->out.dtype == HERO_I8 || is_fp16ish(a->out.dtype), HERO_ERR_UNSUPPORTED, "out dtype %d", a->out.dtype);
  if (a->out.dtype == HERO_I8)
    HERO_REQUIRE((a->out.gran == HERO_GRAN_FWQ || a->out.gran == HERO_GRAN_SQ) && a->out.scale, HERO_ERR_UNSUPPORTED,
                 "INT8 X_attn is feature-wise (FWQ) or static (SQ) with a calibrated scale (Sec. 2.2.2)");
  HERO_REQUIRE(a->s_q > 0 && a->s_k > 0 && a->s_v > 0 && a->s_p > 0, HERO_ERR_INVALID_ARG, "scales must be positive");
  HERO_REQUIRE(a->mask == HERO_MASK_NONE || a->mask == HERO_MASK_CAUSAL, HERO_ERR_INVALID_ARG, "unknown mask %d", a->mask);
  HERO_REQUIRE((int64_t)a->S * 255 * 127 < (1ll << 31), HERO_ERR_UNSUPPORTED, "S=%d would overflow the INT32 accumulator", a->S);
  if (a->B == 0) return HERO_OK;

  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->B; p.S = a->S; p.nh = a->nh; p.dh = a->dh;
  p.nqt = (a->S + ATT_BM - 1) / ATT_BM;
  p.c2 = (float)((double)a->s_q * (double)a->s_k / sqrt((double)a->dh) * 1.4426950408889634);
  p.inv_sp = 1.0f / a->s_p;
  p.pv_scale = a->s_p * a->s_v;
  p.out_scale = a->out.dtype == HERO_I8 ? a->out.scale : nullptr;
  p.out_scale_stride = a->out.gran == HERO_GRAN_FWQ ? 1 : 0;
  p.mask = a->mask; p.key_len = a->key_len;
  p.out = a->out.data; p.out_ld = a->out.ld; p.out_dt = a->out.dtype;
  p.err = h->d_error;
  HERO_REQUIRE((long long)p.nqt * a->nh * a->B < (1ll << 31), HERO_ERR_UNSUPPORTED, "too many tiles");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (a->dh == 64) return launch_attn<64>(h, a, p, s);
  return launch_attn<128>(h, a, p, s);
}
