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
// Persistent: one CTA per SM walks the (batch, head, 128-query tile) list; the K / V / Q rings and the score
// buffers keep running across tile boundaries, so the next tile's operands load and its first Q K^T issues while
// the current tile's epilogue is still draining.  18 warps:
//   warps 0-15 softmax / epilogue: row r = 32 * (w % 4) + lane, columns 32 * (w / 4) .. +31 of a block
//   warp  16   TMA producer (Q once, K per block and sweep, V per block in sweep 2)
//   warp  17   UMMA issuer (one lane) and owner of the TMEM allocation
// The exponentials are the binding resource (16 per clock per SM against 8192 INT8 MACs), so every other
// conversion stays off that unit: INT32 scores become floats by an integer add into a float's mantissa
// and an exact subtraction, and P_u8 is rounded by adding 1.5 * 2^23 inside an FMA.
// TMEM: three score buffers of 128 columns (the UMMA issuer runs two blocks ahead of the softmax warps, which
// hides the issue -> commit -> barrier -> tcgen05.ld round trip) + dh output columns.
#include "attention_common.cuh"

namespace hero {

template <int DH>
struct AttnCfg {
  static constexpr int TILE = ATT_BM * DH;                     // bytes of a Q / K / V tile (INT8)
  static constexpr int P_TILE = ATT_BM * ATT_BN;               // bytes of a P_u8 tile
  static constexpr int KST = (DH == 64) ? 6 : 4;               // K ring depth (TMA latency ~ several block times)
  static constexpr int VST = (DH == 64) ? 4 : 3;               // V ring depth
  static constexpr int OFF_K = 2 * TILE;                       // Q is double-buffered across tiles
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_P = OFF_V + VST * TILE;
  static constexpr int OFF_STATS = OFF_P + 2 * P_TILE;         // float2 [2][4][128]
  static constexpr int OFF_BARS = OFF_STATS + 2 * 4 * ATT_BM * 8;
  static constexpr int NBARS = 4 + 2 * KST + 2 * VST + 2 * ATT_NSB + 4 + 2;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + NBARS * 8 + 16;
  static constexpr uint32_t SWZ = (DH == 128) ? ptx::SWZ_128B : ptx::SWZ_64B;
  static constexpr uint32_t SBO = 8 * DH;                      // 8 rows of DH bytes
  static constexpr int TMEM_COLS = 512;
  static constexpr int O_COL = ATT_NSB * ATT_BN;
};

// ROWMAX: P quantized against the row maximum (see attention_resident.cu): sweep 1 then only finds the maximum of the
// integer scores, sweep 2 does the one exponential per score and sums the un-quantized exponentials.
// F8: e4m3 Q, K, V and an e4m3 P (the FP8 variant): kind::f8f6f4 MMAs, FP32 scores and accumulator, static s_p.
// PROBE: also writes the raw scores, the P codes and the raw accumulators to global memory (verification only).
template <int DH, bool ROWMAX, bool F8 = false, bool PROBE = false>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_int8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using Cfg = AttnCfg<DH>;
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
  uint64_t* s_full = v_empty + VST;             // [ATT_NSB]
  uint64_t* s_empty = s_full + ATT_NSB;         // [ATT_NSB]  one arrival per softmax warp
  uint64_t* p_full = s_empty + ATT_NSB;               // [2]  one arrival per softmax warp
  uint64_t* p_empty = p_full + 2;               // [2]
  uint64_t* o_full = p_empty + 2;               // [1]
  uint64_t* o_empty = o_full + 1;               // [1]  one arrival per softmax warp
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.nqt * p.nh * p.B;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 1);
      ptx::mbar_init(&p_full[i], ATT_SM_WARPS); ptx::mbar_init(&p_empty[i], 1);
    }
    for (int i = 0; i < ATT_NSB; ++i) { ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_empty[i], ATT_SM_WARPS); }
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
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();                                       // the previous kernel's outputs are complete and visible from here on

  if (warp == ATT_TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer
    // The rings run on across tile boundaries, so the next tile's Q and first K blocks are already in
    // flight while the softmax warps finish the current tile.
    // (The helper loops are walked by the whole warp, one elected lane issuing: with uniform control flow the addresses
    // stay in the uniform datapath; ring positions advance without divisions.  A helper's turn-around time is part of
    // every hand-off.)
    {
      const bool issue = ptx::elect_one();
      RingPos<KST> kr;
      RingPos<VST> vr;
      uint32_t wcnt = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int row_base = b * p.S, col0 = h * DH;
        const int qb = wcnt & 1;
        if (!ptx::mbar_wait(&q_empty[qb], ((wcnt >> 1) & 1) ^ 1, p.err, 0x1000 | qb)) { ok = false; break; }
        if (issue) {
          ptx::mbar_expect_tx(&q_full[qb], Cfg::TILE);
          ptx::tma_load_2d(sQ + qb * Cfg::TILE, &tmQ, col0, row_base + qt * ATT_BM, &q_full[qb]);
        }
        for (int i = 0; i < 2 * nkv; ++i) {
          const int j = i < nkv ? i : i - nkv;
          const int ks = kr.idx;
          if (!ptx::mbar_wait(&k_empty[ks], kr.par ^ 1, p.err, 0x1100 | ks)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&k_full[ks], Cfg::TILE);
            ptx::tma_load_2d(sK + ks * Cfg::TILE, &tmK, col0, row_base + j * ATT_BN, &k_full[ks]);
          }
          kr.advance(1);
          if (i >= nkv) {
            const int vs = vr.idx;
            if (!ptx::mbar_wait(&v_empty[vs], vr.par ^ 1, p.err, 0x1200 | vs)) { ok = false; break; }
            if (issue) {
              ptx::mbar_expect_tx(&v_full[vs], Cfg::TILE);
              ptx::tma_load_2d(sV + vs * Cfg::TILE, &tmV, col0, row_base + j * ATT_BN, &v_full[vs]);
            }
            vr.advance(1);
          }
        }
        ++wcnt;
      }
    }
    __syncwarp();
  } else if (warp == ATT_MMA_WARP) {
    // ------------------------------------------------------------------ UMMA issuer
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // Q, K: K-major rows of DH bytes
      constexpr uint64_t pmaj = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);      // P: K-major rows of 128 bytes
      constexpr uint64_t vmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // V: MN-major, 8-key groups
      // descriptors differ only in the start-address field (address >> 4): one base per operand, small additions later
      const uint64_t qd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sQ)), kd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sK));
      const uint64_t pd0 = ptx::smem_desc(pmaj, ptx::smem_u32(sP)), vd0 = ptx::smem_desc(vmaj, ptx::smem_u32(sV));
      RingPos<KST> kr;
      RingPos<VST> vr;
      RingPos<ATT_NSB> sr;
      uint32_t pcnt = 0, wcnt = 0;
      bool ok = true;

      auto issue_pv = [&](int j) -> bool {
        if (j == 0 && !ptx::mbar_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x2500)) return false;   // previous tile's O read out
        const int vs = vr.idx, pb = pcnt & 1;
        if (!ptx::mbar_wait(&v_full[vs], vr.par, p.err, 0x2100 | vs)) return false;
        if (!ptx::mbar_wait(&p_full[pb], (pcnt >> 1) & 1, p.err, 0x2200 | pb)) return false;
        ptx::tc_fence_after();
        if (issue) {
          const uint64_t pd = pd0 + (uint32_t)((pb * Cfg::P_TILE) >> 4), vd = vd0 + (uint32_t)((vs * Cfg::TILE) >> 4);
#pragma unroll
          for (int k = 0; k < ATT_BN / 32; ++k)
            if constexpr (F8) ptx::umma_f8(tmem_base + Cfg::O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (j | k) != 0);
            else ptx::umma_i8(tmem_base + Cfg::O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (j | k) != 0);
          ptx::umma_commit(&v_empty[vs]);
          ptx::umma_commit(&p_empty[pb]);
        }
        vr.advance(1); ++pcnt;
        return true;
      };

      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int qb = wcnt & 1;
        if (!ptx::mbar_wait(&q_full[qb], (wcnt >> 1) & 1, p.err, 0x2000 | qb)) { ok = false; break; }
        const uint64_t qd = qd0 + (uint32_t)((qb * Cfg::TILE) >> 4);
        for (int i = 0; i < 2 * nkv && ok; ++i) {
          const int ks = kr.idx, sb = sr.idx;
          if (!ptx::mbar_wait(&k_full[ks], kr.par, p.err, 0x2300 | ks)) { ok = false; break; }
          if (!ptx::mbar_wait(&s_empty[sb], sr.par ^ 1, p.err, 0x2400 | sb)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint64_t kd = kd0 + (uint32_t)((ks * Cfg::TILE) >> 4);
#pragma unroll
            for (int k = 0; k < DH / 32; ++k)
              if constexpr (F8) ptx::umma_f8(tmem_base + sb * ATT_BN, qd + 2 * k, kd + 2 * k, p.idesc_qk, k != 0);
              else ptx::umma_i8(tmem_base + sb * ATT_BN, qd + 2 * k, kd + 2 * k, p.idesc_qk, k != 0);
            ptx::umma_commit(&k_empty[ks]);
            ptx::umma_commit(&s_full[sb]);
            if (i == 2 * nkv - 1) ptx::umma_commit(&q_empty[qb]);   // Q buffer free once these MMAs have read it
          }
          kr.advance(1); sr.advance(1);
          if (i >= nkv + 1) ok = issue_pv(i - nkv - 1);
        }
        if (ok) ok = issue_pv(nkv - 1);
        if (ok && issue) ptx::umma_commit(o_full);
        ++wcnt;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    const int quarter = warp & 3, cq = warp >> 2;            // TMEM lane quarter, 32-column group of a block
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;
    uint32_t scnt = 0, pcnt = 0, wcnt = 0;
    bool ok = true;

    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      int qt, h, b, klen; attn_tile(p, t, qt, h, b);
      const int nkv = attn_nkv(p, qt, b, klen);
      const int q0 = qt * ATT_BM, row_base = b * p.S, col0 = h * DH;
      const int q = q0 + r_loc;
      const bool row_ok = q < p.S;
      int kmax = klen - 1;                                   // last allowed key (inclusive)
      if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);

      // verification outputs: row (b, h, q) of the [B*nh][S][S] score / code arrays
      const long long probe_row = ((long long)(b * p.nh + h) * p.S + q) * p.S;
      auto probe_scores = [&](const uint32_t (&r)[32], int key0) {
        if constexpr (PROBE) {
          if (p.dbg_scores && row_ok) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (key0 + e < p.S) p.dbg_scores[probe_row + key0 + e] = (int)r[e];
          }
        }
      };

      float m = -INFINITY, l = 0.f;
      if constexpr (ROWMAX) {
        // ---- sweep 1: row maximum of the integer scores only
        int imax = -(1 << 21);                               // below every real score
        for (int i = 0; i < nkv; ++i, ++scnt) {
          const int sb = scnt % ATT_NSB;
          if (ok && !ptx::mbar_wait(&s_full[sb], (scnt / ATT_NSB) & 1, p.err, 0x3000 | sb)) ok = false;
          ptx::tc_fence_after();
          {
            uint32_t r[32];
            ptx::tmem_ld32(t_lane + sb * ATT_BN + cq * 32, r);
            ptx::tmem_ld_wait();
            probe_scores(r, i * ATT_BN + cq * 32);
            const int nvalid = min(32, kmax - (i * ATT_BN + cq * 32) + 1);
            if (nvalid < 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j) if (j >= nvalid) r[j] = (uint32_t)(-(1 << 21));
            }
            int i0 = max((int)r[0], (int)r[1]), i1 = max((int)r[2], (int)r[3]);
#pragma unroll
            for (int j = 4; j < 32; j += 4) { i0 = max(i0, max((int)r[j], (int)r[j + 1])); i1 = max(i1, max((int)r[j + 2], (int)r[j + 3])); }
            imax = max(imax, max(i0, i1));
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&s_empty[sb]);
        }
        m = (float)imax;
      } else {
      // ---- sweep 1: running row max and row sum (log2 domain)
      for (int i = 0; i < nkv; ++i, ++scnt) {
        const int sb = scnt % ATT_NSB;
        if (ok && !ptx::mbar_wait(&s_full[sb], (scnt / ATT_NSB) & 1, p.err, 0x3000 | sb)) ok = false;
        ptx::tc_fence_after();
        {
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + cq * 32, r);
          ptx::tmem_ld_wait();
          const int kb = i * ATT_BN + cq * 32;
          probe_scores(r, kb);
          const int nvalid = min(32, kmax - kb + 1);       // keys kb .. kb + nvalid - 1 are allowed
          if (nvalid > 0) {
            float m_blk;
            if constexpr (F8) {
              float fm = -INFINITY;
#pragma unroll
              for (int j = 0; j < 32; ++j) fm = fmaxf(fm, j < nvalid ? __uint_as_float(r[j]) : -INFINITY);
              m_blk = fm * c2;
            } else {
            int imax = INT_MIN;
            if (nvalid == 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j) imax = max(imax, (int)r[j]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) imax = max(imax, j < nvalid ? (int)r[j] : INT_MIN);
            }
              m_blk = (float)imax * c2;
            }
            const float m_new = fmaxf(m, m_blk);
            float2 acc2 = make_float2(0.f, 0.f);
            const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m_new, -m_new), mg = make_float2(-ATT_MAGIC, -ATT_MAGIC);
            if constexpr (F8) {
#pragma unroll
              for (int j = 0; j < 32; ++j) acc2.x += j < nvalid ? ex2f(fmaf(__uint_as_float(r[j]), c2, -m_new)) : 0.f;
            } else if (nvalid == 32) {
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const float2 f = __fadd2_rn(make_float2(__uint_as_float(0x4B400000u + r[j]), __uint_as_float(0x4B400000u + r[j + 1])), mg);
                const float2 tt = __ffma2_rn(f, c22, nm2);
                acc2 = __fadd2_rn(acc2, make_float2(ex2f(tt.x), ex2f(tt.y)));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) acc2.x += j < nvalid ? ex2f(fmaf(score_to_float(r[j]), c2, -m_new)) : 0.f;
            }
            l = l * ex2f(m - m_new) + (acc2.x + acc2.y);    // m = -inf on first use: 2^-inf = 0
            m = m_new;
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_empty[sb]);
      }
      }
      // ---- combine the four column groups of each row (buffer alternates with the tile)
      float2* st = stats + (wcnt & 1) * 4 * ATT_BM;
      st[cq * ATT_BM + r_loc] = make_float2(m, l);
      asm volatile("bar.sync 1, 512;" ::: "memory");
      float pscale;
      if constexpr (ROWMAX) {
        float mf = st[r_loc].x;
#pragma unroll
        for (int g = 1; g < 4; ++g) mf = fmaxf(mf, st[g * ATT_BM + r_loc].x);
        m = mf <= (float)(-(1 << 21)) ? INFINITY : mf * c2;   // no allowed key: every exponential becomes exactly 0
        pscale = 255.0f;                                      // P~_u8 = Round(255 * 2^(t - m))
      } else {
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
        // P_u8 = Round(P / s_p) with P = 2^(t - m) / l
        pscale = l > 0.f ? p.inv_sp / l : 0.f;
      }

      // ---- sweep 2: scores again -> P_u8 in shared memory (UMMA K-major, 128-byte swizzle)
      for (int j = 0; j < nkv; ++j, ++scnt, ++pcnt) {
        const int sb = scnt % ATT_NSB, pb = pcnt & 1;
        if (ok && !ptx::mbar_wait(&s_full[sb], (scnt / ATT_NSB) & 1, p.err, 0x3100 | sb)) ok = false;
        if (ok && !ptx::mbar_wait(&p_empty[pb], ((pcnt >> 1) & 1) ^ 1, p.err, 0x3200 | pb)) ok = false;
        ptx::tc_fence_after();
        {
          const uint32_t prow = ptx::smem_u32(sP + pb * Cfg::P_TILE) + (r_loc >> 3) * 1024 + (r_loc & 7) * 128;
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + cq * 32, r);
          ptx::tmem_ld_wait();
          const int kb = j * ATT_BN + cq * 32;
          const int nvalid = min(32, kmax - kb + 1);
          float y[32];
          const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m, -m), mg = make_float2(-ATT_MAGIC, -ATT_MAGIC);
          const float2 ps2 = make_float2(pscale, pscale), rm2 = make_float2(ATT_MAGIC, ATT_MAGIC);
          if constexpr (ROWMAX) {
            if (nvalid < 32) {                                 // masked keys: 2^(very negative) = 0, in P~ and in the row sum
#pragma unroll
              for (int e = 0; e < 32; ++e) if (e >= nvalid) r[e] = (uint32_t)(-(1 << 21));
            }
            float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float2 tt = __ffma2_rn(make_float2((float)(int)r[e], (float)(int)r[e + 1]), c22, nm2);
              const float2 ev = make_float2(ex2f(tt.x), ex2f(tt.y));
              acc2 = __fadd2_rn(acc2, ev);
              const float2 v = __ffma2_rn(ev, ps2, rm2);       // at most 255: no clip
              y[e] = v.x; y[e + 1] = v.y;
            }
            l += acc2.x + acc2.y;
          } else if constexpr (F8) {
            // P / s_p as a float; the conversion to e4m3 (saturating at 448, round to nearest even) happens at the pack
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float2 tt = __ffma2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), c22, nm2);
              const float2 v = __fmul2_rn(make_float2(ex2f(tt.x), ex2f(tt.y)), ps2);
              y[e] = e < nvalid ? v.x : 0.f;
              y[e + 1] = e + 1 < nvalid ? v.y : 0.f;
            }
          } else {
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            // Round(P / s_p) clipped to 255: round-half-to-even happens in the FMA's single rounding
            const float2 f = __fadd2_rn(make_float2(__uint_as_float(0x4B400000u + r[e]), __uint_as_float(0x4B400000u + r[e + 1])), mg);
            const float2 tt = __ffma2_rn(f, c22, nm2);
            const float2 v = __ffma2_rn(make_float2(ex2f(tt.x), ex2f(tt.y)), ps2, rm2);
            y[e] = fminf(v.x, ATT_MAGIC + 255.0f);
            y[e + 1] = fminf(v.y, ATT_MAGIC + 255.0f);
          }
          if (nvalid < 32) {                                   // block straddles the mask: masked keys get code 0
#pragma unroll
            for (int e = 0; e < 32; ++e) if (e >= nvalid) y[e] = ATT_MAGIC;
          }
          }
          const int c16 = cq * 2;                              // 16-byte chunk index within the 128-byte row
          if constexpr (PROBE) {
            if (p.dbg_p && row_ok) {
#pragma unroll
              for (int e = 0; e < 32; ++e) if (kb + e < p.S) p.dbg_p[probe_row + kb + e] = (uint8_t)(__float_as_uint(y[e]) & 0xffu);
            }
          }
          if constexpr (F8) {
            st_shared16(prow + (((c16) ^ (r_loc & 7)) << 4), ptx::f32x4_to_e4m3x4(y[0], y[1], y[2], y[3]),
                        ptx::f32x4_to_e4m3x4(y[4], y[5], y[6], y[7]), ptx::f32x4_to_e4m3x4(y[8], y[9], y[10], y[11]),
                        ptx::f32x4_to_e4m3x4(y[12], y[13], y[14], y[15]));
            st_shared16(prow + (((c16 + 1) ^ (r_loc & 7)) << 4), ptx::f32x4_to_e4m3x4(y[16], y[17], y[18], y[19]),
                        ptx::f32x4_to_e4m3x4(y[20], y[21], y[22], y[23]), ptx::f32x4_to_e4m3x4(y[24], y[25], y[26], y[27]),
                        ptx::f32x4_to_e4m3x4(y[28], y[29], y[30], y[31]));
          } else {
          st_shared16(prow + (((c16) ^ (r_loc & 7)) << 4), low_bytes4_u(y[0], y[1], y[2], y[3]), low_bytes4_u(y[4], y[5], y[6], y[7]),
                      low_bytes4_u(y[8], y[9], y[10], y[11]), low_bytes4_u(y[12], y[13], y[14], y[15]));
          st_shared16(prow + (((c16 + 1) ^ (r_loc & 7)) << 4), low_bytes4_u(y[16], y[17], y[18], y[19]),
                      low_bytes4_u(y[20], y[21], y[22], y[23]), low_bytes4_u(y[24], y[25], y[26], y[27]),
                      low_bytes4_u(y[28], y[29], y[30], y[31]));
          }
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async_smem();                         // generic-proxy writes -> visible to the UMMA (async proxy)
        __syncwarp();
        if (lane == 0) { ptx::mbar_arrive(&s_empty[sb]); ptx::mbar_arrive(&p_full[pb]); }
      }

      float rowf = 1.f;
      if constexpr (ROWMAX) {
        // the row sum across the four column groups (the .y halves of this tile's statistics slots)
        reinterpret_cast<float*>(st)[2 * (cq * ATT_BM + r_loc) + 1] = l;
        asm volatile("bar.sync 1, 512;" ::: "memory");
        float lt = 0.f;
#pragma unroll
        for (int g = 0; g < 4; ++g) lt += reinterpret_cast<const float*>(st)[2 * (g * ATT_BM + r_loc) + 1];
        rowf = lt > 0.f ? 1.0f / lt : 0.f;
      }
      // ---- epilogue: X_attn = acc * s_p s_v (/ S_attn[j] -> Round -> INT8); 32 output columns per warp
      uint32_t r[32];
      if (nkv > 0) {
        if (ok && !ptx::mbar_wait(o_full, wcnt & 1, p.err, 0x3300)) ok = false;
        ptx::tc_fence_after();
        if (cq * 32 < DH) {
          ptx::tmem_ld32(t_lane + Cfg::O_COL + cq * 32, r);
          ptx::tmem_ld_wait();
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(o_empty);              // the accumulator may be overwritten by the next tile
        ++wcnt;
      }
      if (nkv == 0) {
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = 0;                 // every key masked: the row is zero
      }
      if (cq * 32 < DH && row_ok) {
        const int ocol = cq * 32;
        const long long grow = (long long)(row_base + q);
        const int gcol = col0 + ocol;
        if constexpr (PROBE) {
          if (p.dbg_acc) {
#pragma unroll
            for (int j = 0; j < 32; ++j) p.dbg_acc[grow * ((long long)p.nh * p.dh) + gcol + j] = (int)r[j];
          }
        }
        auto accf = [&](int j) -> float { return F8 ? __uint_as_float(r[j]) : (float)(int)r[j]; };
        if (p.out_dt == HERO_F8) {
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j)
            v[j] = accf(j) * rowf * (p.pv_scale / __ldg(p.out_scale + (gcol + j) * p.out_scale_stride));
          uint8_t* dst = reinterpret_cast<uint8_t*>(p.out) + grow * p.out_ld + gcol;
#pragma unroll
          for (int g = 0; g < 2; ++g)
            st_g16(dst + 16 * g, ptx::f32x4_to_e4m3x4(v[16 * g], v[16 * g + 1], v[16 * g + 2], v[16 * g + 3]),
                   ptx::f32x4_to_e4m3x4(v[16 * g + 4], v[16 * g + 5], v[16 * g + 6], v[16 * g + 7]),
                   ptx::f32x4_to_e4m3x4(v[16 * g + 8], v[16 * g + 9], v[16 * g + 10], v[16 * g + 11]),
                   ptx::f32x4_to_e4m3x4(v[16 * g + 12], v[16 * g + 13], v[16 * g + 14], v[16 * g + 15]));
        } else if (p.out_dt == HERO_I8) {
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j)
            v[j] = accf(j) * rowf * (p.pv_scale / __ldg(p.out_scale + (gcol + j) * p.out_scale_stride));
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
            for (int e = 0; e < 8; ++e) v[e] = accf(8 * g + e) * rowf * p.pv_scale;
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

template <int DH, bool ROWMAX, bool F8 = false, bool PROBE = false>
static hero_status launch_attn(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = AttnCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  CUtensorMap tq, tk, tv;
  hero_status st;
  if ((st = make_tmap_2d(h, &tq, a->q, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BM, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if (F8) {
    p.idesc_qk = ptx::make_idesc(1, 0, 0, 0, 0, ATT_BM, ATT_BN); // E4M3 x E4M3 -> F32, both K-major
    p.idesc_pv = ptx::make_idesc(1, 0, 0, 0, 1, ATT_BM, DH);     // E4M3 x E4M3 -> F32, V is MN-major
  } else {
    p.idesc_qk = ptx::make_idesc(2, 1, 1, 0, 0, ATT_BM, ATT_BN); // S8 x S8 -> S32, both K-major
    p.idesc_pv = ptx::make_idesc(2, 0, 1, 0, 1, ATT_BM, DH);     // U8 x S8 -> S32, V is MN-major
  }
  auto kern = attn_int8_kernel<DH, ROWMAX, F8, PROBE>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  const long long tiles = (long long)p.nqt * a->nh * a->B;
  const int grid = (int)(tiles < h->sm_count ? tiles : h->sm_count);   // persistent: one CTA per SM
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(ATT_THREADS), Cfg::SMEM_BYTES, stream, tq, tk, tv, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero

namespace hero {
static hero_status attention_impl(hero_handle* h, const hero_attn_args* a, const hero_attn_probe* probe, void* stream) {
  HERO_REQUIRE(h && a, HERO_ERR_INVALID_ARG, "hero_int8_attention: NULL handle or args");
  HERO_REQUIRE(a->q && a->k && a->v, HERO_ERR_INVALID_ARG, "q, k, v are required");
  HERO_REQUIRE(a->B >= 0 && a->S > 0 && a->nh > 0, HERO_ERR_INVALID_ARG, "bad B / S / nh");
  HERO_REQUIRE(a->dh == 64 || a->dh == 128, HERO_ERR_UNSUPPORTED, "dh=%d: 64 or 128 supported", a->dh);
  const bool fp_in = is_fp16ish(a->dtype), f8_in = a->dtype == HERO_F8;
  HERO_REQUIRE(a->dtype == HERO_I8 || f8_in || fp_in, HERO_ERR_UNSUPPORTED, "q/k/v dtype %d: INT8, e4m3, F16 or BF16 expected", a->dtype);
  HERO_REQUIRE(!f8_in || a->p_mode == HERO_P_STATIC, HERO_ERR_UNSUPPORTED, "the e4m3 core quantizes P with the static scale only");
  HERO_REQUIRE(!f8_in || a->out.dtype != HERO_I8, HERO_ERR_UNSUPPORTED, "the e4m3 core emits e4m3, F16 or BF16");
  HERO_REQUIRE(a->out.dtype != HERO_F8 || f8_in || fp_in, HERO_ERR_UNSUPPORTED, "an e4m3 X_attn needs e4m3 or FP operands");
  HERO_REQUIRE(aligned16(a->q) && aligned16(a->k) && aligned16(a->v) && (a->ld * (fp_in ? 2 : 1)) % 16 == 0 &&
               a->ld >= (int64_t)a->nh * a->dh,
               HERO_ERR_ALIGNMENT, "q/k/v must be 16-byte aligned with a row pitch that is a multiple of 16 bytes and ld >= nh*dh");
  hero_status st;
  if ((st = check_matrix(a->out, "out")) != HERO_OK) return st;
  HERO_REQUIRE(a->out.rows == (int64_t)a->B * a->S && a->out.cols == (int64_t)a->nh * a->dh, HERO_ERR_INVALID_ARG,
               "out must be [B*S, nh*dh]");
  HERO_REQUIRE(is_q8(a->out.dtype) || is_fp16ish(a->out.dtype), HERO_ERR_UNSUPPORTED, "out dtype %d", a->out.dtype);
  HERO_REQUIRE(!(fp_in && a->out.dtype == HERO_F8), HERO_ERR_UNSUPPORTED, "the FP16 / BF16 core emits INT8, F16 or BF16");
  if (is_q8(a->out.dtype))
    HERO_REQUIRE((a->out.gran == HERO_GRAN_FWQ || a->out.gran == HERO_GRAN_SQ) && a->out.scale, HERO_ERR_UNSUPPORTED,
                 "INT8 X_attn is feature-wise (FWQ) or static (SQ) with a calibrated scale (Sec. 2.2.2)");
  HERO_REQUIRE(fp_in || (a->s_q > 0 && a->s_k > 0 && a->s_v > 0 && (a->s_p > 0 || a->p_mode == HERO_P_ROWMAX)), HERO_ERR_INVALID_ARG, "scales must be positive");
  HERO_REQUIRE(a->mask == HERO_MASK_NONE || a->mask == HERO_MASK_CAUSAL, HERO_ERR_INVALID_ARG, "unknown mask %d", a->mask);
  HERO_REQUIRE(fp_in || (int64_t)a->S * 255 * 127 < (1ll << 31), HERO_ERR_UNSUPPORTED, "S=%d would overflow the INT32 accumulator", a->S);
  if (a->B == 0) return HERO_OK;

  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->B; p.S = a->S; p.nh = a->nh; p.dh = a->dh;
  p.nqt = (a->S + ATT_BM - 1) / ATT_BM;
  p.c2 = (float)((double)a->s_q * (double)a->s_k / sqrt((double)a->dh) * 1.4426950408889634);
  HERO_REQUIRE(a->p_mode == HERO_P_STATIC || a->p_mode == HERO_P_ROWMAX, HERO_ERR_INVALID_ARG, "unknown p_mode %d", a->p_mode);
  const bool rowmax = !fp_in && a->p_mode == HERO_P_ROWMAX;
  p.inv_sp = rowmax ? 255.0f : 1.0f / a->s_p;
  p.pv_scale = rowmax ? a->s_v / 255.0f : a->s_p * a->s_v;
  p.out_scale = is_q8(a->out.dtype) ? a->out.scale : nullptr;
  p.out_scale_stride = a->out.gran == HERO_GRAN_FWQ ? 1 : 0;
  p.mask = a->mask; p.key_len = a->key_len;
  p.out = a->out.data; p.out_ld = a->out.ld; p.out_dt = a->out.dtype;
  p.err = h->d_error;
  p.p_absmax = a->p_absmax;
  HERO_REQUIRE(a->p_absmax == nullptr || fp_in, HERO_ERR_UNSUPPORTED, "p_absmax is observed by the F16 / BF16 attention core only");
  p.obs_col = a->out_col_absmax;
  HERO_REQUIRE(a->out_col_absmax == nullptr || (fp_in && is_fp16ish(a->out.dtype)), HERO_ERR_UNSUPPORTED,
               "out_col_absmax is observed by the F16 / BF16 attention core on an F16 / BF16 output only");
  HERO_REQUIRE((long long)p.nqt * a->nh * a->B < (1ll << 31), HERO_ERR_UNSUPPORTED, "too many tiles");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (probe) {
    HERO_REQUIRE(a->dtype == HERO_I8, HERO_ERR_UNSUPPORTED, "the verification outputs exist for the INT8 core only");
    p.dbg_scores = probe->scores; p.dbg_p = probe->p_codes; p.dbg_acc = probe->acc;
    if (a->S <= 512) return (a->dh == 128 && a->S > 384 ? attn_resident_dispatch : attn_pipe_dispatch)(h, a, p, s, true);
    if (rowmax) return a->dh == 64 ? launch_attn<64, true, false, true>(h, a, p, s) : launch_attn<128, true, false, true>(h, a, p, s);
    return a->dh == 64 ? launch_attn<64, false, false, true>(h, a, p, s) : launch_attn<128, false, false, true>(h, a, p, s);
  }
  if (fp_in) return attn_fp_dispatch(h, a, p, s);
  // the score row fits tensor memory (INT8 or e4m3): the pipelined kernel, except for the one shape whose row and
  // accumulator together exceed it there (dh = 128 with more than 384 keys)
  if (a->S <= 512) return (a->dh == 128 && a->S > 384 ? attn_resident_dispatch : attn_pipe_dispatch)(h, a, p, s, false);
  if (f8_in) return a->dh == 64 ? launch_attn<64, false, true>(h, a, p, s) : launch_attn<128, false, true>(h, a, p, s);
  if (rowmax) return a->dh == 64 ? launch_attn<64, true>(h, a, p, s) : launch_attn<128, true>(h, a, p, s);
  if (a->dh == 64) return launch_attn<64, false>(h, a, p, s);
  return launch_attn<128, false>(h, a, p, s);
}
}  // namespace hero

extern "C" hero_status hero_int8_attention(hero_handle* h, const hero_attn_args* a, void* stream) {
  return hero::attention_impl(h, a, nullptr, stream);
}

extern "C" hero_status hero_int8_attention_probe(hero_handle* h, const hero_attn_args* a, const hero_attn_probe* probe,
                                                 void* stream) {
  HERO_REQUIRE(probe != nullptr, HERO_ERR_INVALID_ARG, "hero_int8_attention_probe: probe is NULL");
  return hero::attention_impl(h, a, probe, stream);
}
