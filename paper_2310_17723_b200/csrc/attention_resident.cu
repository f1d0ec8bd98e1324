// INT8 attention core (Sec. 2.2.2 Eq. 15-17) for sequences of at most 512 keys: the whole score row lives in
// tensor memory.  Q K^T is issued once for all (up to four) 128-key blocks into the 512 TMEM columns; the softmax
// warps turn each 32-column piece into e = 2^(t - m_piece) with the piece's own maximum, write e back over the
// scores and keep (m_piece, sum) in registers; once the row maximum and sum are known every piece is re-read,
// scaled by 2^(m_piece - m) / (l s_p) -- one multiply, no second exponential -- rounded to P_u8 and stored as the
// UMMA operand of P V.  One exponential per score instead of two, no second Q K^T pass, K loaded once.  The output
// accumulator aliases the first score block's columns: P V for block 0 is issued only after every warp has consumed
// that block.
#include "attention_common.cuh"

namespace hero {

constexpr int RES_NB = 4;    // score blocks resident in TMEM (4 x 128 columns)

template <int DH>
struct AttnResCfg {
  static constexpr int TILE = ATT_BM * DH;
  static constexpr int P_TILE = ATT_BM * ATT_BN;
  static constexpr int KST = (DH == 64) ? 6 : 4;
  static constexpr int VST = (DH == 64) ? 4 : 3;
  static constexpr int OFF_K = 2 * TILE;
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_P = OFF_V + VST * TILE;
  static constexpr int OFF_STATS = OFF_P + 2 * P_TILE;
  static constexpr int OFF_BARS = OFF_STATS + 2 * 4 * ATT_BM * 8;
  static constexpr int NBARS = 4 + 2 * KST + 2 * VST + 2 * RES_NB + 4 + 2;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + NBARS * 8 + 16;
  static constexpr uint32_t SWZ = (DH == 128) ? ptx::SWZ_128B : ptx::SWZ_64B;
  static constexpr uint32_t SBO = 8 * DH;
  static constexpr int TMEM_COLS = 512;
};

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_int8_resident_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                          const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using Cfg = AttnResCfg<DH>;
  constexpr int KST = Cfg::KST, VST = Cfg::VST;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + Cfg::OFF_K;
  uint8_t* sV = smem + Cfg::OFF_V;
  uint8_t* sP = smem + Cfg::OFF_P;
  float2* stats = reinterpret_cast<float2*>(smem + Cfg::OFF_STATS);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BARS);
  uint64_t* q_full = bars;                      // [2]
  uint64_t* q_empty = q_full + 2;               // [2]
  uint64_t* k_full = q_empty + 2;               // [KST]
  uint64_t* k_empty = k_full + KST;             // [KST]
  uint64_t* v_full = k_empty + KST;             // [VST]
  uint64_t* v_empty = v_full + VST;             // [VST]
  uint64_t* s_full = v_empty + VST;             // [RES_NB]  scores of block j written
  uint64_t* s_free = s_full + RES_NB;           // [RES_NB]  block j consumed by every softmax warp
  uint64_t* p_full = s_free + RES_NB;           // [2]
  uint64_t* p_empty = p_full + 2;               // [2]
  uint64_t* o_full = p_empty + 2;               // [1]
  uint64_t* o_empty = o_full + 1;               // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.nqt * p.nh * p.B;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 1);
      ptx::mbar_init(&p_full[i], ATT_SM_WARPS); ptx::mbar_init(&p_empty[i], 1);
    }
    for (int i = 0; i < RES_NB; ++i) { ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_free[i], ATT_SM_WARPS); }
    for (int i = 0; i < KST; ++i) { ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < VST; ++i) { ptx::mbar_init(&v_full[i], 1); ptx::mbar_init(&v_empty[i], 1); }
    ptx::mbar_init(o_full, 1); ptx::mbar_init(o_empty, ATT_SM_WARPS);
    ptx::fence_mbar_init();
  }
  if (warp == ATT_MMA_WARP) { ptx::tmem_alloc(tmem_slot, Cfg::TMEM_COLS); ptx::tmem_relinquish(); }
  if (warp == ATT_TMA_WARP && lane == 0) { ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == ATT_TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer: Q, every K block, every V block
    if (lane == 0) {
      uint32_t kcnt = 0, vcnt = 0, wcnt = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int row_base = b * p.S, col0 = h * DH;
        const int qb = wcnt & 1;
        if (!ptx::mbar_wait(&q_empty[qb], ((wcnt >> 1) & 1) ^ 1, p.err, 0x7000 | qb)) { ok = false; break; }
        ptx::mbar_expect_tx(&q_full[qb], Cfg::TILE);
        ptx::tma_load_2d(sQ + qb * Cfg::TILE, &tmQ, col0, row_base + qt * ATT_BM, &q_full[qb]);
        for (int j = 0; j < nkv && ok; ++j, ++kcnt) {
          const int ks = kcnt % KST;
          if (!ptx::mbar_wait(&k_empty[ks], ((kcnt / KST) & 1) ^ 1, p.err, 0x7100 | ks)) { ok = false; break; }
          ptx::mbar_expect_tx(&k_full[ks], Cfg::TILE);
          ptx::tma_load_2d(sK + ks * Cfg::TILE, &tmK, col0, row_base + j * ATT_BN, &k_full[ks]);
        }
        for (int j = 0; j < nkv && ok; ++j, ++vcnt) {
          const int vs = vcnt % VST;
          if (!ptx::mbar_wait(&v_empty[vs], ((vcnt / VST) & 1) ^ 1, p.err, 0x7200 | vs)) { ok = false; break; }
          ptx::mbar_expect_tx(&v_full[vs], Cfg::TILE);
          ptx::tma_load_2d(sV + vs * Cfg::TILE, &tmV, col0, row_base + j * ATT_BN, &v_full[vs]);
        }
        ++wcnt;
      }
    }
    __syncwarp();
  } else if (warp == ATT_MMA_WARP) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);
      constexpr uint64_t pmaj = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);
      constexpr uint64_t vmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);
      uint32_t kcnt = 0, vcnt = 0, pcnt = 0, wcnt = 0;
      uint32_t used[RES_NB] = {0, 0, 0, 0};               // how often each score block has been filled so far
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int qb = wcnt & 1;
        if (!ptx::mbar_wait(&q_full[qb], (wcnt >> 1) & 1, p.err, 0x8000 | qb)) { ok = false; break; }
        const uint32_t q_addr = ptx::smem_u32(sQ + qb * Cfg::TILE);
        // the output accumulator of the previous tile sits in block 0's columns: it must have been read out
        if (!ptx::mbar_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x8500)) { ok = false; break; }
#pragma unroll
        for (int j = 0; j < RES_NB; ++j) {
          if (j < nkv && ok) {
            const int ks = kcnt % KST;
            if (!ptx::mbar_wait(&k_full[ks], (kcnt / KST) & 1, p.err, 0x8300 | ks)) { ok = false; }
            if (ok && !ptx::mbar_wait(&s_free[j], (used[j] & 1) ^ 1, p.err, 0x8400 | j)) { ok = false; }
            if (ok) {
              ptx::tc_fence_after();
              const uint32_t k_addr = ptx::smem_u32(sK + ks * Cfg::TILE);
#pragma unroll
              for (int k = 0; k < DH / 32; ++k)
                ptx::umma_i8(tmem_base + j * ATT_BN, ptx::smem_desc(kmaj, q_addr + k * 32),
                             ptx::smem_desc(kmaj, k_addr + k * 32), p.idesc_qk, k != 0);
              ptx::umma_commit(&k_empty[ks]);
              ptx::umma_commit(&s_full[j]);
              ++kcnt; ++used[j];
            }
          }
        }
        if (ok) ptx::umma_commit(&q_empty[qb]);
        for (int j = 0; j < nkv && ok; ++j) {
          const int vs = vcnt % VST, pb = pcnt & 1;
          if (!ptx::mbar_wait(&v_full[vs], (vcnt / VST) & 1, p.err, 0x8100 | vs)) { ok = false; break; }
          if (!ptx::mbar_wait(&p_full[pb], (pcnt >> 1) & 1, p.err, 0x8200 | pb)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t p_addr = ptx::smem_u32(sP + pb * Cfg::P_TILE);
          const uint32_t v_addr = ptx::smem_u32(sV + vs * Cfg::TILE);
#pragma unroll
          for (int k = 0; k < ATT_BN / 32; ++k)
            ptx::umma_i8(tmem_base, ptx::smem_desc(pmaj, p_addr + k * 32), ptx::smem_desc(vmaj, v_addr + k * 32 * DH),
                         p.idesc_pv, (j | k) != 0);
          ptx::umma_commit(&v_empty[vs]);
          ptx::umma_commit(&p_empty[pb]);
          ++vcnt; ++pcnt;
        }
        if (ok) ptx::umma_commit(o_full);
        ++wcnt;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    const int quarter = warp & 3, cq = warp >> 2;            // TMEM lane quarter, 32-column piece of every block
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;
    uint32_t pcnt = 0, wcnt = 0;
    uint32_t used[RES_NB] = {0, 0, 0, 0};
    bool ok = true;

    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      int qt, h, b, klen; attn_tile(p, t, qt, h, b);
      const int nkv = attn_nkv(p, qt, b, klen);
      const int q0 = qt * ATT_BM, row_base = b * p.S, col0 = h * DH;
      const int q = q0 + r_loc;
      const bool row_ok = q < p.S;
      int kmax = klen - 1;
      if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);

      // ---- sweep 1: per piece, e = 2^(t - m_piece) written back over the scores; (m_piece, sum) kept
      float mj[RES_NB], lj[RES_NB];
#pragma unroll
      for (int j = 0; j < RES_NB; ++j) {
        mj[j] = -INFINITY; lj[j] = 0.f;
        if (j < nkv) {
          if (ok && !ptx::mbar_wait(&s_full[j], used[j] & 1, p.err, 0x9000 | j)) ok = false;
          ptx::tc_fence_after();
          if (ok) {
            uint32_t r[32];
            const uint32_t ta = t_lane + j * ATT_BN + cq * 32;
            ptx::tmem_ld32(ta, r);
            ptx::tmem_ld_wait();
            const int kb = j * ATT_BN + cq * 32;
            const int nvalid = min(32, kmax - kb + 1);
            if (nvalid > 0) {
              int imax = INT_MIN;
              if (nvalid == 32) {
#pragma unroll
                for (int e = 0; e < 32; ++e) imax = max(imax, (int)r[e]);
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) imax = max(imax, e < nvalid ? (int)r[e] : INT_MIN);
              }
              const float m = (float)imax * c2;
              float2 acc2 = make_float2(0.f, 0.f);
              const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m, -m), mg = make_float2(-ATT_MAGIC, -ATT_MAGIC);
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                const float2 f = __fadd2_rn(make_float2(__uint_as_float(0x4B400000u + r[e]), __uint_as_float(0x4B400000u + r[e + 1])), mg);
                const float2 tt = __ffma2_rn(f, c22, nm2);
                float2 ev = make_float2(ex2f(tt.x), ex2f(tt.y));
                if (nvalid < 32) { if (e >= nvalid) ev.x = 0.f; if (e + 1 >= nvalid) ev.y = 0.f; }
                acc2 = __fadd2_rn(acc2, ev);
                r[e] = __float_as_uint(ev.x); r[e + 1] = __float_as_uint(ev.y);
              }
              mj[j] = m; lj[j] = acc2.x + acc2.y;
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) r[e] = 0;         // every key of the piece masked
            }
            ptx::tmem_st32(ta, r);
          }
        }
      }
      if (ok) ptx::tmem_st_wait();
      // ---- row maximum and sum: first over this thread's pieces, then across the four column groups
      float m = -INFINITY, l = 0.f;
#pragma unroll
      for (int j = 0; j < RES_NB; ++j) m = fmaxf(m, mj[j]);
#pragma unroll
      for (int j = 0; j < RES_NB; ++j) if (mj[j] > -INFINITY) l += lj[j] * ex2f(mj[j] - m);
      float2* st = stats + (wcnt & 1) * 4 * ATT_BM;
      st[cq * ATT_BM + r_loc] = make_float2(m, l);
      asm volatile("bar.sync 1, 512;" ::: "memory");
      {
        float mf = -INFINITY;
#pragma unroll
        for (int g = 0; g < 4; ++g) mf = fmaxf(mf, st[g * ATT_BM + r_loc].x);
        float lf = 0.f;
        if (mf > -INFINITY) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const float2 o = st[g * ATT_BM + r_loc];
            if (o.x > -INFINITY) lf += o.y * ex2f(o.x - mf);
          }
        }
        m = mf; l = lf;
      }
      const float pscale = l > 0.f ? p.inv_sp / l : 0.f;

      // ---- sweep 2: P_u8 = Round(e * 2^(m_piece - m) / (l s_p)), clipped to 255, into the UMMA operand tile
#pragma unroll
      for (int j = 0; j < RES_NB; ++j) {
        if (j < nkv) {
          const int pb = pcnt & 1;
          if (ok && !ptx::mbar_wait(&p_empty[pb], ((pcnt >> 1) & 1) ^ 1, p.err, 0x9200 | pb)) ok = false;
          if (ok) {
            const uint32_t prow = ptx::smem_u32(sP + pb * Cfg::P_TILE) + (r_loc >> 3) * 1024 + (r_loc & 7) * 128;
            uint32_t r[32];
            ptx::tmem_ld32(t_lane + j * ATT_BN + cq * 32, r);
            ptx::tmem_ld_wait();
            const float f = mj[j] > -INFINITY ? ex2f(mj[j] - m) * pscale : 0.f;
            const float2 f2v = make_float2(f, f), rm2 = make_float2(ATT_MAGIC, ATT_MAGIC);
            float y[32];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float2 v = __ffma2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v, rm2);
              y[e] = fminf(v.x, ATT_MAGIC + 255.0f);
              y[e + 1] = fminf(v.y, ATT_MAGIC + 255.0f);
            }
            const int c16 = cq * 2;
            st_shared16(prow + (((c16) ^ (r_loc & 7)) << 4), low_bytes4_u(y[0], y[1], y[2], y[3]), low_bytes4_u(y[4], y[5], y[6], y[7]),
                        low_bytes4_u(y[8], y[9], y[10], y[11]), low_bytes4_u(y[12], y[13], y[14], y[15]));
            st_shared16(prow + (((c16 + 1) ^ (r_loc & 7)) << 4), low_bytes4_u(y[16], y[17], y[18], y[19]),
                        low_bytes4_u(y[20], y[21], y[22], y[23]), low_bytes4_u(y[24], y[25], y[26], y[27]),
                        low_bytes4_u(y[28], y[29], y[30], y[31]));
          }
          ptx::tc_fence_before();
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) { ptx::mbar_arrive(&s_free[j]); ptx::mbar_arrive(&p_full[pb]); }
          ++pcnt; ++used[j];
        }
      }

      // ---- epilogue: X_attn = acc * s_p s_v (/ S_attn[j] -> Round -> INT8); the accumulator sits in columns 0 .. DH-1
      uint32_t r[32];
      if (nkv > 0) {
        if (ok && !ptx::mbar_wait(o_full, wcnt & 1, p.err, 0x9300)) ok = false;
        ptx::tc_fence_after();
        if (ok && cq * 32 < DH) {
          ptx::tmem_ld32(t_lane + cq * 32, r);
          ptx::tmem_ld_wait();
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(o_empty);
        ++wcnt;
      }
      if (nkv == 0 || !ok) {
#pragma unroll
        for (int e = 0; e < 32; ++e) r[e] = 0;
      }
      if (cq * 32 < DH && row_ok) {
        const long long grow = (long long)(row_base + q);
        const int gcol = col0 + cq * 32;
        if (p.out_dt == HERO_I8) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e)
            v[e] = (float)(int)r[e] * (p.pv_scale / __ldg(p.out_scale + (gcol + e) * p.out_scale_stride));
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
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == ATT_MMA_WARP) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int DH>
static hero_status launch_resident(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = AttnResCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  CUtensorMap tq, tk, tv;
  hero_status st;
  if ((st = make_tmap_2d(h, &tq, a->q, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BM, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  p.idesc_qk = ptx::make_idesc(2, 1, 1, 0, 0, ATT_BM, ATT_BN);
  p.idesc_pv = ptx::make_idesc(2, 0, 1, 0, 1, ATT_BM, DH);
  auto kern = attn_int8_resident_kernel<DH>;
  static bool configured = false;
  if (!configured) {
    HERO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES));
    configured = true;
  }
  const long long tiles = (long long)p.nqt * a->nh * a->B;
  const int grid = (int)(tiles < h->sm_count ? tiles : h->sm_count);
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    kern<<<grid, ATT_THREADS, Cfg::SMEM_BYTES, stream>>>(tq, tk, tv, p);
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

hero_status attn_resident_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  if (a->dh == 64) return launch_resident<64>(h, a, p, stream);
  return launch_resident<128>(h, a, p, stream);
}

}  // namespace hero
