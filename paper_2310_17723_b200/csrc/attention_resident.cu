// INT8 attention core (Sec. 2.2.2 Eq. 15-17) for sequences of at most 512 keys: the whole score row lives in
// tensor memory.  Q K^T is issued once for all (up to four) 128-key blocks into the 512 TMEM columns; the softmax
// warps turn each 32-column piece into e = 2^(t - m_piece) with the piece's own maximum, write e back over the
// scores and keep a running (max, sum); once the row maximum and sum are known every piece is re-read, scaled by
// 2^(m_piece - m) / (l s_p) -- one multiply, no second exponential -- rounded to P_u8 and stored as the UMMA operand
// of P V.  One exponential per score instead of two, no second Q K^T pass, K loaded once.
//
// The output accumulator occupies the columns of score block 3 (columns 384 ..).  With at most three key blocks it
// is a buffer of its own.  With four, block 3 is converted to P first (the P V order is 3, 0, 1, 2), so its columns
// are free when the first P V lands there, and the next tile's Q K^T for block 3 waits until the previous output
// has been read.  The epilogue of tile t runs inside tile t+1, after the first three score blocks of t+1 have been
// exponentiated: P V of tile t finishes in the shadow of that work.
#include "attention_common.cuh"
#include <type_traits>

namespace hero {


constexpr int RES_NB = 4;          // score blocks resident in TMEM (4 x 128 columns)
constexpr int RES_O_COL = 384;     // output accumulator columns
constexpr int RES_NP = 3;          // P operand tiles in shared memory

// the j-th block in P V order
__device__ __forceinline__ int res_pv_block(int nkv, int i) { return nkv == RES_NB ? ((i + 3) & 3) : i; }

template <int DH>
struct AttnResCfg {
  static constexpr int TILE = ATT_BM * DH;
  static constexpr int P_TILE = ATT_BM * ATT_BN;
  static constexpr int KST = (DH == 64) ? 6 : 4;
  static constexpr int VST = (DH == 64) ? 4 : 3;
  static constexpr int OFF_K = 2 * TILE;
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_P = OFF_V + VST * TILE;
  static constexpr int OFF_STATS = OFF_P + RES_NP * P_TILE;
  static constexpr int OFF_PM = OFF_STATS + 2 * 4 * ATT_BM * 8;        // per-thread piece maxima [RES_NB][512] x 2 halves
  static constexpr int OFF_OSC = OFF_PM + RES_NB * 512 * 8;            // per-tile output factors [lane quarter][2][128]
  static constexpr int OFF_BARS = OFF_OSC + 4 * 2 * 128 * 4;
  static constexpr int NBARS = 4 + 2 * KST + 2 * VST + 2 * RES_NB + 2 * RES_NP + 2;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + NBARS * 8 + 16;
  static constexpr uint32_t SWZ = (DH == 128) ? ptx::SWZ_128B : ptx::SWZ_64B;
  static constexpr uint32_t SBO = 8 * DH;
  static constexpr int TMEM_COLS = 512;
};

// X_attn = acc * s_p s_v (/ S_attn[j] -> Round -> INT8) for the tile whose P V has been issued; frees the accumulator
// columns.  Every softmax warp takes DH / 4 columns of its 32 rows; `osc` is the tile's per-column factor
// s_p s_v / S_attn[j] (s_p s_v alone for an FP output) staged in shared memory.  Kept out of line: it runs once per
// tile and its registers stay out of the sweeps' allocation.
template <int DH, bool F8, bool PROBE>
__device__ __noinline__ void res_epilogue(const AttnParams& p, uint32_t t_lane, uint64_t* o_full, uint64_t* o_empty,
                                          uint32_t parity, int cq, int lane, long long pend_row, int pend_col,
                                          const float* osc, float rowf, bool& ok) {
  constexpr int CW = DH / 4;
  uint32_t r[CW];
  // A wait that gives up has recorded its code; the warp then runs on without waiting again (what it computes no
  // longer matters, every access stays in bounds) so that the kernel ends promptly.
  if (ok && !ptx::mbar_wait(o_full, parity, p.err, 0x9300)) ok = false;
  ptx::tc_fence_after();
  if constexpr (CW == 16) ptx::tmem_ld16(t_lane + RES_O_COL + cq * CW, r);
  else ptx::tmem_ld32(t_lane + RES_O_COL + cq * CW, r);
  ptx::tmem_ld_wait();
  ptx::tc_fence_before();
  __syncwarp();
  if (lane == 0) ptx::mbar_arrive(o_empty);
  if (pend_row >= 0) {
    const int gcol = pend_col + cq * CW;
    if constexpr (PROBE) {
      if (p.dbg_acc) {
        int* dst = p.dbg_acc + pend_row * ((long long)p.nh * p.dh) + gcol;
#pragma unroll
        for (int c = 0; c < CW; ++c) dst[c] = (int)r[c];
      }
    }
    const float4* o4 = reinterpret_cast<const float4*>(osc + cq * CW);
    auto acc = [&](int c) -> float { if constexpr (F8) return __uint_as_float(r[c]); else return (float)(int)r[c]; };
    if (p.out_dt == HERO_F8) {
      // e4m3 X_attn (FP8 variant): the conversion saturates and rounds to nearest even
      int8_t* dst = reinterpret_cast<int8_t*>(p.out) + pend_row * p.out_ld + gcol;
#pragma unroll
      for (int g = 0; g < CW / 16; ++g) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float4 sc = o4[4 * g + k];
          const int c = 16 * g + 4 * k;
          w[k] = ptx::f32x4_to_e4m3x4(acc(c) * rowf * sc.x, acc(c + 1) * rowf * sc.y, acc(c + 2) * rowf * sc.z, acc(c + 3) * rowf * sc.w);
        }
        st_g16(dst + 16 * g, w[0], w[1], w[2], w[3]);
      }
    } else if (p.out_dt == HERO_I8) {
      int8_t* dst = reinterpret_cast<int8_t*>(p.out) + pend_row * p.out_ld + gcol;
#pragma unroll
      for (int g = 0; g < CW / 16; ++g) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float4 sc = o4[4 * g + k];
          const int c = 16 * g + 4 * k;
          const float a = fminf(fmaxf((float)(int)r[c] * rowf * sc.x, -127.f), 127.f) + ATT_MAGIC;
          const float b = fminf(fmaxf((float)(int)r[c + 1] * rowf * sc.y, -127.f), 127.f) + ATT_MAGIC;
          const float cc = fminf(fmaxf((float)(int)r[c + 2] * rowf * sc.z, -127.f), 127.f) + ATT_MAGIC;
          const float d = fminf(fmaxf((float)(int)r[c + 3] * rowf * sc.w, -127.f), 127.f) + ATT_MAGIC;
          w[k] = low_bytes4_u(a, b, cc, d);                  // low byte of magic + x = two's-complement Round(x)
        }
        st_g16(dst + 16 * g, w[0], w[1], w[2], w[3]);
      }
    } else {
      uint16_t* dst = reinterpret_cast<uint16_t*>(p.out) + pend_row * p.out_ld + gcol;
#pragma unroll
      for (int g = 0; g < CW / 8; ++g) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = acc(8 * g + e) * rowf * p.pv_scale;
        st_g16(dst + 8 * g, fp2(v[0], v[1], p.out_dt), fp2(v[2], v[3], p.out_dt), fp2(v[4], v[5], p.out_dt),
               fp2(v[6], v[7], p.out_dt));
      }
    }
  }
}

// ROWMAX: the long-sequence-robust P quantizer (not in the paper): P~_u8 = Round(255 * 2^(t - m_row)) with the row sum
// l of the un-quantized 2^(t - m_row) kept in FP32 and divided out in the epilogue.  Sweep 1 then only finds the row
// maximum (integer compares, nothing written back), sweep 2 does the one exponential per score.
// F8: e4m3 Q, K, V and an e4m3 P (the FP8 variant; static P quantizer only): kind::f8f6f4 products, FP32 scores and
// accumulator in tensor memory, P formed by the saturating conversion instead of round + clip.
// PROBE: also writes the raw scores, the P codes and the raw accumulators to global memory (verification only).
template <int DH, bool ROWMAX, bool F8, bool PROBE>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_int8_resident_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                          const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnParams p) {
  using Cfg = AttnResCfg<DH>;
  constexpr int KST = Cfg::KST, VST = Cfg::VST;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + Cfg::OFF_K;
  uint8_t* sV = smem + Cfg::OFF_V;
  uint8_t* sP = smem + Cfg::OFF_P;
  float2* stats = reinterpret_cast<float2*>(smem + Cfg::OFF_STATS);
  float2* pm2 = reinterpret_cast<float2*>(smem + Cfg::OFF_PM) + (threadIdx.x & 511);
  float* osc_s = reinterpret_cast<float*>(smem + Cfg::OFF_OSC);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BARS);
  uint64_t* q_full = bars;                      // [2]
  uint64_t* q_empty = q_full + 2;               // [2]
  uint64_t* k_full = q_empty + 2;               // [KST]
  uint64_t* k_empty = k_full + KST;             // [KST]
  uint64_t* v_full = k_empty + KST;             // [VST]
  uint64_t* v_empty = v_full + VST;             // [VST]
  uint64_t* s_full = v_empty + VST;             // [RES_NB]  scores of block j written
  uint64_t* s_free = s_full + RES_NB;           // [RES_NB]  block j consumed by every softmax warp
  uint64_t* p_full = s_free + RES_NB;           // [RES_NP]
  uint64_t* p_empty = p_full + RES_NP;          // [RES_NP]
  uint64_t* o_full = p_empty + RES_NP;          // [1]
  uint64_t* o_empty = o_full + 1;               // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.nqt * p.nh * p.B;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 1); }
    for (int i = 0; i < RES_NP; ++i) { ptx::mbar_init(&p_full[i], ATT_SM_WARPS); ptx::mbar_init(&p_empty[i], 1); }
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
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();                                       // the previous kernel's outputs are complete and visible from here on

  if (warp == ATT_TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer: Q, K blocks, V blocks in P V order
    // (helper loops: whole warp, one elected lane issues, ring positions without divisions; see attention.cu)
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
        if (!ptx::mbar_wait(&q_empty[qb], ((wcnt >> 1) & 1) ^ 1, p.err, 0x7000 | qb)) { ok = false; break; }
        if (issue) {
          ptx::mbar_expect_tx(&q_full[qb], Cfg::TILE);
          ptx::tma_load_2d(sQ + qb * Cfg::TILE, &tmQ, col0, row_base + qt * ATT_BM, &q_full[qb]);
        }
        for (int j = 0; j < nkv && ok; ++j, kr.advance(1)) {
          const int ks = kr.idx;
          if (!ptx::mbar_wait(&k_empty[ks], kr.par ^ 1, p.err, 0x7100 | ks)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&k_full[ks], Cfg::TILE);
            ptx::tma_load_2d(sK + ks * Cfg::TILE, &tmK, col0, row_base + j * ATT_BN, &k_full[ks]);
          }
        }
        for (int i = 0; i < nkv && ok; ++i, vr.advance(1)) {
          const int j = res_pv_block(nkv, i);
          const int vs = vr.idx;
          if (!ptx::mbar_wait(&v_empty[vs], vr.par ^ 1, p.err, 0x7200 | vs)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&v_full[vs], Cfg::TILE);
            ptx::tma_load_2d(sV + vs * Cfg::TILE, &tmV, col0, row_base + j * ATT_BN, &v_full[vs]);
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
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);
      constexpr uint64_t pmaj = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);
      constexpr uint64_t vmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);
      const uint64_t qd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sQ)), kd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sK));
      const uint64_t pd0 = ptx::smem_desc(pmaj, ptx::smem_u32(sP)), vd0 = ptx::smem_desc(vmaj, ptx::smem_u32(sV));
      RingPos<KST> kr;
      RingPos<VST> vr;
      RingPos<RES_NP> pr;
      uint32_t wcnt = 0;
      uint32_t used = 0;                                  // bit j: parity of how often score block j has been filled
      bool ok = true;

      // S_j = Q K_j^T of the tile with running index w into score block j.  K stages are consumed in issue order,
      // which the callers keep equal to the producer's order j = 0, 1, ...
      auto issue_qk = [&](uint32_t w, int j) {
        const int qb = w & 1;
        const int ks = kr.idx;
        if (!ptx::mbar_wait(&k_full[ks], kr.par, p.err, 0x8300 | ks)) { ok = false; return; }
        if (!ptx::mbar_wait(&s_free[j], ((used >> j) & 1) ^ 1, p.err, 0x8400 | j)) { ok = false; return; }
        ptx::tc_fence_after();
        if (issue) {
          const uint64_t qd = qd0 + (uint32_t)((qb * Cfg::TILE) >> 4), kd = kd0 + (uint32_t)((ks * Cfg::TILE) >> 4);
#pragma unroll
          for (int k = 0; k < DH / 32; ++k) {
            if constexpr (F8) ptx::umma_f8(tmem_base + j * ATT_BN, qd + 2 * k, kd + 2 * k, p.idesc_qk, k != 0);
            else ptx::umma_i8(tmem_base + j * ATT_BN, qd + 2 * k, kd + 2 * k, p.idesc_qk, k != 0);
          }
          ptx::umma_commit(&k_empty[ks]);
          ptx::umma_commit(&s_full[j]);
        }
        kr.advance(1); used ^= 1u << j;
      };
      // next tile of this CTA with at least one key block
      auto next_tile = [&](int t, int& nkv) {
        for (; t < total_tiles; t += gridDim.x) {
          int qt, h, b, klen; attn_tile(p, t, qt, h, b);
          nkv = attn_nkv(p, qt, b, klen);
          if (nkv > 0) return t;
        }
        nkv = 0;
        return total_tiles;
      };

      int nkv = 0, nkv_n = 0;
      int t = next_tile(blockIdx.x, nkv);
      int issued = 0;                                     // leading score blocks of the current tile already issued
      bool q_ready = false;                               // q_full of the current tile already awaited
      while (t < total_tiles && ok) {
        const int tn = next_tile(t + gridDim.x, nkv_n);
        const int qb = wcnt & 1;
        if (!q_ready && !ptx::mbar_wait(&q_full[qb], (wcnt >> 1) & 1, p.err, 0x8000 | qb)) { ok = false; break; }
        bool o_free = false;                              // previous tile's output read out of columns 384 ..
        for (int j = issued; j < nkv && ok; ++j) {
          if (j == 3) {
            if (!ptx::mbar_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x8500)) { ok = false; break; }
            o_free = true;
          }
          issue_qk(wcnt, j);
        }
        if (!ok) break;
        if (issue) ptx::umma_commit(&q_empty[qb]);
        issued = 0; q_ready = false;
        for (int i = 0; i < nkv && ok; ++i) {
          const int vs = vr.idx, pb = pr.idx;
          if (!ptx::mbar_wait(&v_full[vs], vr.par, p.err, 0x8100 | vs)) { ok = false; break; }
          if (!ptx::mbar_wait(&p_full[pb], pr.par, p.err, 0x8200 | pb)) { ok = false; break; }
          if (!o_free) {
            if (!ptx::mbar_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x8600)) { ok = false; break; }
            o_free = true;
          }
          ptx::tc_fence_after();
          if (issue) {
            const uint64_t pd = pd0 + (uint32_t)((pb * Cfg::P_TILE) >> 4), vd = vd0 + (uint32_t)((vs * Cfg::TILE) >> 4);
#pragma unroll
            for (int k = 0; k < ATT_BN / 32; ++k) {
              if constexpr (F8) ptx::umma_f8(tmem_base + RES_O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (i | k) != 0);
              else ptx::umma_i8(tmem_base + RES_O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (i | k) != 0);
            }
            ptx::umma_commit(&v_empty[vs]);
            ptx::umma_commit(&p_empty[pb]);
          }
          vr.advance(1); pr.advance(1);
          // the block just converted to P is free: start the next tile's scores there (block 3 holds the output)
          const int j = res_pv_block(nkv, i);
          if (j == issued && j < 3 && j < nkv_n) {
            if (!q_ready) {
              const uint32_t wn = wcnt + 1;
              if (!ptx::mbar_wait(&q_full[wn & 1], (wn >> 1) & 1, p.err, 0x8700)) { ok = false; break; }
              q_ready = true;
            }
            issue_qk(wcnt + 1, j);
            ++issued;
          }
        }
        if (ok && issue) ptx::umma_commit(o_full);
        ++wcnt;
        t = tn; nkv = nkv_n;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    const int quarter = warp & 3, cq = warp >> 2;            // TMEM lane quarter, 32-column piece of every block
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;
    uint32_t pcnt = 0, wcnt = 0, used = 0;
    bool ok = true;
    long long pend_row = -1;                                 // output row of the tile whose epilogue is pending
    int pend_col = 0;
    float pend_rowf = 1.f;
    bool pend = false;

    auto epilogue = [&]() {
      res_epilogue<DH, F8, PROBE>(p, t_lane, o_full, o_empty, (wcnt - 1) & 1, cq, lane, pend_row, pend_col,
                       osc_s + quarter * 256 + ((wcnt - 1) & 1) * 128, pend_rowf, ok);
      pend = false;
    };

    // the next tile's coordinates are decoded one iteration ahead: the integer divisions and the key-length load
    // overlap the current tile's work instead of standing at the head of every iteration
    int qt_n = 0, h_n = 0, b_n = 0, klen_n = 0, nkv_n = 0;
    if ((int)blockIdx.x < total_tiles) { attn_tile(p, blockIdx.x, qt_n, h_n, b_n); nkv_n = attn_nkv(p, qt_n, b_n, klen_n); }
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      const int qt = qt_n, h = h_n, b = b_n, klen = klen_n, nkv = nkv_n;
      if (t + (int)gridDim.x < total_tiles) { attn_tile(p, t + gridDim.x, qt_n, h_n, b_n); nkv_n = attn_nkv(p, qt_n, b_n, klen_n); }
      const int q0 = qt * ATT_BM, row_base = b * p.S, col0 = h * DH;
      const int q = q0 + r_loc;
      const bool row_ok = q < p.S;
      float osc_raw = 1.f;                                   // this thread's S_attn[j], turned into a factor further down
      if (is_q8(p.out_dt) && cq * 32 + lane < DH)
        osc_raw = __ldg(p.out_scale + (long long)(col0 + cq * 32 + lane) * p.out_scale_stride);
      if (nkv == 0) {
        // every key masked: the rows are zero, no tensor work
        if (cq * 32 < DH && row_ok) {
          const long long grow = (long long)(row_base + q);
          const int gcol = col0 + cq * 32;
          const int es = is_q8(p.out_dt) ? 1 : 2;
          uint8_t* dst = reinterpret_cast<uint8_t*>(p.out) + (grow * p.out_ld + gcol) * es;
          for (int g = 0; g < 2 * es; ++g) st_g16(dst + 16 * g, 0u, 0u, 0u, 0u);
        }
        continue;
      }
      int kmax = klen - 1;
      if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);
      // verification outputs: row (b, h, q) of the [B*nh][S][S] score / code arrays
      const long long probe_row = ((long long)(b * p.nh + h) * p.S + q) * p.S;
      auto probe_scores = [&](const uint32_t (&r)[16], int key0) {
        if constexpr (PROBE) {
          if (p.dbg_scores && row_ok) {
#pragma unroll
            for (int e = 0; e < 16; ++e) if (key0 + e < p.S) p.dbg_scores[probe_row + key0 + e] = (int)r[e];
          }
        }
      };
      auto probe_codes = [&](const uint32_t (&w)[4], int key0) {
        if constexpr (PROBE) {
          if (p.dbg_p && row_ok) {
#pragma unroll
            for (int e = 0; e < 16; ++e) if (key0 + e < p.S) p.dbg_p[probe_row + key0 + e] = (uint8_t)(w[e >> 2] >> (8 * (e & 3)));
          }
        }
      };

      float m = -INFINITY, l = 0.f;
      if constexpr (ROWMAX) {
        // ---- sweep 1: the row maximum of the integer scores (the scale d~ log2 e is positive); nothing is written back
        int imax = -(1 << 21);                               // below every real score (|t| <= 127^2 * 128 < 2^21)
#pragma unroll 1
        for (int j = 0; j < nkv; ++j) {
          if (j == 3 && pend) epilogue();                    // block 3's columns hold the previous tile's output
          if (ok && !ptx::mbar_wait(&s_full[j], (used >> j) & 1, p.err, 0x9000 | j)) ok = false;
          ptx::tc_fence_after();
          const uint32_t ta = t_lane + j * ATT_BN + cq * 32;
          const int kb = j * ATT_BN + cq * 32;
          uint32_t ra[16], rb[16];
          ptx::tmem_ld16(ta, ra);
          ptx::tmem_ld16(ta + 16, rb);
          ptx::tmem_ld_wait();
          probe_scores(ra, kb); probe_scores(rb, kb + 16);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t (&r)[16] = hh ? rb : ra;
            const int nvalid = min(16, kmax - (kb + 16 * hh) + 1);
            if (nvalid < 16) {
#pragma unroll
              for (int e = 0; e < 16; ++e) if (e >= nvalid) r[e] = (uint32_t)(-(1 << 21));
            }
            int i0 = max((int)r[0], (int)r[1]), i1 = max((int)r[2], (int)r[3]);
#pragma unroll
            for (int e = 4; e < 16; e += 4) { i0 = max(i0, max((int)r[e], (int)r[e + 1])); i1 = max(i1, max((int)r[e + 2], (int)r[e + 3])); }
            imax = max(imax, max(i0, i1));
          }
        }
        m = (float)imax;                                     // exchanged as an (exact) integer-valued float
      } else {
      // ---- sweep 1: per piece, e = 2^(t - m_piece) written back over the scores; running (m, l) in registers.
      // FULL: every key of every block is valid for every row of the tile (no mask, no short sequence): the loop then
      // carries no per-piece validity logic at all.
      auto sweep1 = [&](auto full_tag) {
      constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll 1
      for (int j = 0; j < nkv; ++j) {
        if (j == 3 && pend) epilogue();                      // block 3's columns hold the previous tile's output
        if (ok && !ptx::mbar_wait(&s_full[j], (used >> j) & 1, p.err, 0x9000 | j)) ok = false;
        ptx::tc_fence_after();
        {
          const uint32_t ta = t_lane + j * ATT_BN + cq * 32;
          const int kb = j * ATT_BN + cq * 32;
          float mpa[2];
          uint32_t ra[16], rb[16];
          ptx::tmem_ld16(ta, ra);
          ptx::tmem_ld16(ta + 16, rb);
          ptx::tmem_ld_wait();
          probe_scores(ra, kb); probe_scores(rb, kb + 16);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {                   // two 16-column pieces, each with its own maximum
            uint32_t (&r)[16] = hh ? rb : ra;
            const int nvalid = FULL ? 16 : min(16, kmax - (kb + 16 * hh) + 1);
            float mp = -INFINITY;
            if (FULL || nvalid > 0) {
              if (!FULL && nvalid < 16) {
                // masked keys: a score far below every real one (|t| < 2^21) turns into e = 0 by itself
#pragma unroll
                for (int e = 0; e < 16; ++e) if (e >= nvalid) r[e] = F8 ? __float_as_uint(-1.0e30f) : (uint32_t)(-(1 << 21));
              }
              if constexpr (F8) {
                float f0 = fmaxf(__uint_as_float(r[0]), __uint_as_float(r[1])), f1 = fmaxf(__uint_as_float(r[2]), __uint_as_float(r[3]));
#pragma unroll
                for (int e = 4; e < 16; e += 4) {
                  f0 = fmaxf(f0, fmaxf(__uint_as_float(r[e]), __uint_as_float(r[e + 1])));
                  f1 = fmaxf(f1, fmaxf(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])));
                }
                mp = fmaxf(f0, f1) * c2;
              } else {
                int i0 = max((int)r[0], (int)r[1]), i1 = max((int)r[2], (int)r[3]);
#pragma unroll
                for (int e = 4; e < 16; e += 4) { i0 = max(i0, max((int)r[e], (int)r[e + 1])); i1 = max(i1, max((int)r[e + 2], (int)r[e + 3])); }
                mp = (float)max(i0, i1) * c2;
              }
              float2 acc2 = make_float2(0.f, 0.f);
              const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-mp, -mp);
#pragma unroll
              for (int e = 0; e < 16; e += 2) {
                const float2 f = F8 ? make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]))
                                    : make_float2((float)(int)r[e], (float)(int)r[e + 1]);
                const float2 tt = __ffma2_rn(f, c22, nm2);
                const float2 ev = make_float2(ex2f(tt.x), ex2f(tt.y));
                acc2 = __fadd2_rn(acc2, ev);
                r[e] = __float_as_uint(ev.x); r[e + 1] = __float_as_uint(ev.y);
              }
              const float mn = fmaxf(m, mp);
              l = l * ex2f(m - mn) + (acc2.x + acc2.y) * ex2f(mp - mn);
              m = mn;
            } else {
#pragma unroll
              for (int e = 0; e < 16; ++e) r[e] = 0;         // every key of the piece masked
            }
            ptx::tmem_st16(ta + 16 * hh, r);
            mpa[hh] = mp;
          }
          pm2[j * 512] = make_float2(mpa[0], mpa[1]);
        }
      }
      };
      if (p.mask != HERO_MASK_CAUSAL && klen >= nkv * ATT_BN) sweep1(std::true_type{}); else sweep1(std::false_type{});
      }
      if constexpr (!ROWMAX) ptx::tmem_st_wait();
      if (pend) epilogue();
      // ---- row maximum and sum across the four column groups
      float2* st = stats + (wcnt & 1) * 4 * ATT_BM;
      st[cq * ATT_BM + r_loc] = make_float2(m, l);
      if (cq * 32 + lane < DH) osc_s[quarter * 256 + (wcnt & 1) * 128 + cq * 32 + lane] = __fdividef(p.pv_scale, osc_raw);
      // the four warps that share these 32 rows (one per column group) meet; the other lane quarters are not involved
      asm volatile("bar.sync %0, 128;" ::"r"(1 + quarter) : "memory");
      float pscale = 0.f;
      if constexpr (ROWMAX) {
        float mf = st[r_loc].x;
#pragma unroll
        for (int g = 1; g < 4; ++g) mf = fmaxf(mf, st[g * ATT_BM + r_loc].x);
        // a row without any allowed key: +inf makes every exponential exactly 0
        m = mf <= (float)(-(1 << 21)) ? INFINITY : mf * c2;
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
        pscale = l > 0.f ? __fdividef(p.inv_sp, l) : 0.f;   // 2 ulp: far below the rounding step of P
      }

      // ---- sweep 2: P_u8 = Round(e * 2^(m_piece - m) / (l s_p)), clipped to 255, into the UMMA operand tile
#pragma unroll 1
      for (int i = 0; i < nkv; ++i) {
        const int j = res_pv_block(nkv, i);
        const int pb = pcnt % RES_NP;
        if (ok && !ptx::mbar_wait(&p_empty[pb], ((pcnt / RES_NP) & 1) ^ 1, p.err, 0x9200 | pb)) ok = false;
        {
          const uint32_t prow = ptx::smem_u32(sP + pb * Cfg::P_TILE) + (r_loc >> 3) * 1024 + (r_loc & 7) * 128;
          const int c16 = cq * 2;
          uint32_t ra[16], rb[16];
          ptx::tmem_ld16(t_lane + j * ATT_BN + cq * 32, ra);
          ptx::tmem_ld16(t_lane + j * ATT_BN + cq * 32 + 16, rb);
          ptx::tmem_ld_wait();
          if constexpr (ROWMAX) {
            // P~_u8 = Round(255 * 2^(t - m)): at most 255, no clip; the un-quantized exponentials are summed for l
            const int kb = j * ATT_BN + cq * 32;
            const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m, -m);
            const float2 s255 = make_float2(255.0f, 255.0f), rm2 = make_float2(ATT_MAGIC, ATT_MAGIC);
            float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int g = 0; g < 2; ++g) {
              uint32_t (&r)[16] = g ? rb : ra;
              const int nvalid = min(16, kmax - (kb + 16 * g) + 1);
              if (nvalid < 16) {
#pragma unroll
                for (int e = 0; e < 16; ++e) if (e >= nvalid) r[e] = (uint32_t)(-(1 << 21));   // 2^(very negative) = 0
              }
              uint32_t w[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const int e = 4 * k;
                const float2 ta = __ffma2_rn(make_float2((float)(int)r[e], (float)(int)r[e + 1]), c22, nm2);
                const float2 tb = __ffma2_rn(make_float2((float)(int)r[e + 2], (float)(int)r[e + 3]), c22, nm2);
                const float2 ea = make_float2(ex2f(ta.x), ex2f(ta.y)), eb = make_float2(ex2f(tb.x), ex2f(tb.y));
                acc2 = __fadd2_rn(acc2, __fadd2_rn(ea, eb));
                const float2 ya = __ffma2_rn(ea, s255, rm2), yb = __ffma2_rn(eb, s255, rm2);
                w[k] = low_bytes4_u(ya.x, ya.y, yb.x, yb.y);
              }
              probe_codes(w, kb + 16 * g);
              st_shared16(prow + (((c16 + g) ^ (r_loc & 7)) << 4), w[0], w[1], w[2], w[3]);
            }
            l += acc2.x + acc2.y;
          } else {
          const float2 mp2 = pm2[j * 512];
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            uint32_t (&r)[16] = g ? rb : ra;
            const float mp = g ? mp2.y : mp2.x;
            const float f = mp > -INFINITY ? ex2f(mp - m) * pscale : 0.f;
            const float2 f2v = make_float2(f, f), rm2 = make_float2(ATT_MAGIC, ATT_MAGIC);
            uint32_t w[4];
            if constexpr (F8) {
              // P_f8 = e4m3(e f): the conversion saturates at 448 (s_p = max P / 448)
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const int e = 4 * k;
                const float2 a = __fmul2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v);
                const float2 c = __fmul2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), f2v);
                w[k] = ptx::f32x4_to_e4m3x4(a.x, a.y, c.x, c.y);
              }
            } else if (f <= 255.25f) {
              // e <= 1 in every piece, so e f cannot round above 255: no clip needed
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const int e = 4 * k;
                const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v, rm2);
                const float2 c = __ffma2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), f2v, rm2);
                w[k] = low_bytes4_u(a.x, a.y, c.x, c.y);
              }
            } else {
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const int e = 4 * k;
                const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v, rm2);
                const float2 c = __ffma2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), f2v, rm2);
                w[k] = low_bytes4_u(fminf(a.x, ATT_MAGIC + 255.0f), fminf(a.y, ATT_MAGIC + 255.0f),
                                    fminf(c.x, ATT_MAGIC + 255.0f), fminf(c.y, ATT_MAGIC + 255.0f));
              }
            }
            probe_codes(w, j * ATT_BN + cq * 32 + 16 * g);
            st_shared16(prow + (((c16 + g) ^ (r_loc & 7)) << 4), w[0], w[1], w[2], w[3]);
          }
          }
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) { ptx::mbar_arrive(&s_free[j]); ptx::mbar_arrive(&p_full[pb]); }
        ++pcnt; used ^= 1u << j;
      }
      if constexpr (ROWMAX) {
        // the row sum across the four column groups (the .y halves of this tile's statistics slots)
        reinterpret_cast<float*>(st)[2 * (cq * ATT_BM + r_loc) + 1] = l;
        asm volatile("bar.sync %0, 128;" ::"r"(1 + quarter) : "memory");
        float lt = 0.f;
#pragma unroll
        for (int g = 0; g < 4; ++g) lt += reinterpret_cast<const float*>(st)[2 * (g * ATT_BM + r_loc) + 1];
        pend_rowf = lt > 0.f ? 1.0f / lt : 0.f;
      }
      pend = true;
      pend_row = row_ok ? (long long)(row_base + q) : -1;
      pend_col = col0;
      ++wcnt;
    }
    if (pend) epilogue();
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == ATT_MMA_WARP) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int DH, bool ROWMAX, bool F8, bool PROBE = false>
static hero_status launch_resident(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = AttnResCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  CUtensorMap tq, tk, tv;
  hero_status st;
  if ((st = make_tmap_2d(h, &tq, a->q, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BM, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BN, DH)) != HERO_OK) return st;
  if (F8) {
    p.idesc_qk = ptx::make_idesc(1, 0, 0, 0, 0, ATT_BM, ATT_BN);   // E4M3 x E4M3 -> F32, both K-major
    p.idesc_pv = ptx::make_idesc(1, 0, 0, 0, 1, ATT_BM, DH);       // E4M3 x E4M3 -> F32, V is MN-major
  } else {
    p.idesc_qk = ptx::make_idesc(2, 1, 1, 0, 0, ATT_BM, ATT_BN);   // S8 x S8 -> S32
    p.idesc_pv = ptx::make_idesc(2, 0, 1, 0, 1, ATT_BM, DH);       // U8 x S8 -> S32
  }
  auto kern = attn_int8_resident_kernel<DH, ROWMAX, F8, PROBE>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  const long long tiles = (long long)p.nqt * a->nh * a->B;
  const int grid = (int)(tiles < h->sm_count ? tiles : h->sm_count);
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(ATT_THREADS), Cfg::SMEM_BYTES, stream, tq, tk, tv, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

hero_status attn_resident_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream, bool probe) {
  if (probe) {                                               // INT8 operands only (checked by the caller)
    if (a->p_mode == HERO_P_ROWMAX)
      return a->dh == 64 ? launch_resident<64, true, false, true>(h, a, p, stream) : launch_resident<128, true, false, true>(h, a, p, stream);
    return a->dh == 64 ? launch_resident<64, false, false, true>(h, a, p, stream) : launch_resident<128, false, false, true>(h, a, p, stream);
  }
  if (a->dtype == HERO_F8) {                               // static P quantizer only (checked by the caller)
    if (a->dh == 64) return launch_resident<64, false, true>(h, a, p, stream);
    return launch_resident<128, false, true>(h, a, p, stream);
  }
  if (a->p_mode == HERO_P_ROWMAX) {
    if (a->dh == 64) return launch_resident<64, true, false>(h, a, p, stream);
    return launch_resident<128, true, false>(h, a, p, stream);
  }
  if (a->dh == 64) return launch_resident<64, false, false>(h, a, p, stream);
  return launch_resident<128, false, false>(h, a, p, stream);
}

}  // namespace hero
