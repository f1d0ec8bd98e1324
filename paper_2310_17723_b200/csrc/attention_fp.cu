// FP16 / BF16 attention for a module the mode table leaves in FP (Sec. 2.3, Table 1; Eq. 9-11):
// P = softmax(Q K^T / sqrt(dh)), X_attn = P V with fp32 accumulation, stored in FP16 / BF16 or, when the
// attention-output linear is INT8, quantized by the calibrated S_attn in the epilogue (no standalone
// quantize kernel).  Same persistent, two-sweep, TMEM-resident structure as the INT8 core for long sequences: kind::f16
// MMAs, fp32 scores, P stored as FP16 / BF16 in the UMMA operand layout.  Nothing here quantizes P with a static scale,
// so the first sweep only needs the row maximum (no exponentials): the second sweep forms e = 2^(t - m) <= 1, sums it in
// FP32 and feeds the UN-normalised e to P V; the row sum is divided out of the accumulator in the epilogue.  One
// exponential per score.  A tile row of 128 features is 256 bytes, i.e. two 128-byte-swizzled sub-tiles.
#include "attention_common.cuh"

namespace hero {

template <int DH>
struct AttnFpCfg {
  static constexpr int SUB = ATT_BM * 128;                     // bytes of one [128 rows x 64 elements] sub-tile
  static constexpr int NSUB = DH / 64;                         // sub-tiles per Q / K / V tile
  static constexpr int TILE = SUB * NSUB;
  static constexpr int P_TILE = 2 * SUB;                       // [128 x 128 keys] FP16
  static constexpr int QB = (DH == 64) ? 2 : 1;                // Q buffers
  static constexpr int KST = (DH == 64) ? 4 : 2;
  static constexpr int VST = (DH == 64) ? 3 : 2;
  static constexpr int PB = (DH == 64) ? 2 : 1;                // P buffers
  static constexpr int OFF_K = QB * TILE;
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_P = OFF_V + VST * TILE;
  static constexpr int OFF_STATS = OFF_P + PB * P_TILE;        // float2 [2][4][128]
  static constexpr int OFF_BARS = OFF_STATS + 2 * 4 * ATT_BM * 8;
  static constexpr int NBARS = 2 * QB + 2 * KST + 2 * VST + 2 * ATT_NSB + 2 * PB + 2;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + NBARS * 8 + 16;
  static constexpr int TMEM_COLS = 512;
  static constexpr int O_COL = ATT_NSB * ATT_BN;
};

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_fp_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnParams p, const int in_dt) {
  using Cfg = AttnFpCfg<DH>;
  constexpr int KST = Cfg::KST, VST = Cfg::VST, QB = Cfg::QB, PB = Cfg::PB, NSUB = Cfg::NSUB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + Cfg::OFF_K;
  uint8_t* sV = smem + Cfg::OFF_V;
  uint8_t* sP = smem + Cfg::OFF_P;
  float2* stats = reinterpret_cast<float2*>(smem + Cfg::OFF_STATS);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BARS);
  uint64_t* q_full = bars;                      // [QB]
  uint64_t* q_empty = q_full + QB;              // [QB]
  uint64_t* k_full = q_empty + QB;              // [KST]
  uint64_t* k_empty = k_full + KST;             // [KST]
  uint64_t* v_full = k_empty + KST;             // [VST]
  uint64_t* v_empty = v_full + VST;             // [VST]
  uint64_t* s_full = v_empty + VST;             // [ATT_NSB]
  uint64_t* s_empty = s_full + ATT_NSB;         // [ATT_NSB]
  uint64_t* p_full = s_empty + ATT_NSB;               // [PB]
  uint64_t* p_empty = p_full + PB;              // [PB]
  uint64_t* o_full = p_empty + PB;              // [1]
  uint64_t* o_empty = o_full + 1;               // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.nqt * p.nh * p.B;

  if (threadIdx.x == 0) {
    for (int i = 0; i < QB; ++i) { ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 1); }
    for (int i = 0; i < ATT_NSB; ++i) { ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_empty[i], ATT_SM_WARPS); }
    for (int i = 0; i < PB; ++i) { ptx::mbar_init(&p_full[i], ATT_SM_WARPS); ptx::mbar_init(&p_empty[i], 1); }
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
    // (helper loops: whole warp, one elected lane issues, ring positions without divisions; see attention.cu)
    {
      const bool issue = ptx::elect_one();
      RingPos<KST> kr;
      RingPos<VST> vr;
      RingPos<QB> qr;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int row_base = b * p.S, col0 = h * DH;
        const int qb = qr.idx;
        if (!ptx::mbar_wait(&q_empty[qb], qr.par ^ 1, p.err, 0x4000 | qb)) { ok = false; break; }
        if (issue) {
          ptx::mbar_expect_tx(&q_full[qb], Cfg::TILE);
#pragma unroll
          for (int sIdx = 0; sIdx < NSUB; ++sIdx)
            ptx::tma_load_2d(sQ + qb * Cfg::TILE + sIdx * Cfg::SUB, &tmQ, col0 + sIdx * 64, row_base + qt * ATT_BM, &q_full[qb]);
        }
        for (int i = 0; i < 2 * nkv; ++i) {
          const int j = i < nkv ? i : i - nkv;
          const int ks = kr.idx;
          if (!ptx::mbar_wait(&k_empty[ks], kr.par ^ 1, p.err, 0x4100 | ks)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&k_full[ks], Cfg::TILE);
#pragma unroll
            for (int sIdx = 0; sIdx < NSUB; ++sIdx)
              ptx::tma_load_2d(sK + ks * Cfg::TILE + sIdx * Cfg::SUB, &tmK, col0 + sIdx * 64, row_base + j * ATT_BN, &k_full[ks]);
          }
          kr.advance(1);
          if (i >= nkv) {
            const int vs = vr.idx;
            if (!ptx::mbar_wait(&v_empty[vs], vr.par ^ 1, p.err, 0x4200 | vs)) { ok = false; break; }
            if (issue) {
              ptx::mbar_expect_tx(&v_full[vs], Cfg::TILE);
#pragma unroll
              for (int sIdx = 0; sIdx < NSUB; ++sIdx)
                ptx::tma_load_2d(sV + vs * Cfg::TILE + sIdx * Cfg::SUB, &tmV, col0 + sIdx * 64, row_base + j * ATT_BN, &v_full[vs]);
            }
            vr.advance(1);
          }
        }
        qr.advance(1);
      }
    }
    __syncwarp();
  } else if (warp == ATT_MMA_WARP) {
    // ------------------------------------------------------------------ UMMA issuer
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);          // Q, K, P: K-major, 128-byte rows
      constexpr uint64_t vmaj = ptx::smem_desc_base(Cfg::SUB, 1024, ptx::SWZ_128B);    // V: MN-major; 64-feature chunks SUB apart
      // descriptors differ only in the start-address field (address >> 4): one base per operand, small additions later
      const uint64_t qd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sQ)), kd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sK));
      const uint64_t pd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sP)), vd0 = ptx::smem_desc(vmaj, ptx::smem_u32(sV));
      RingPos<KST> kr;
      RingPos<VST> vr;
      RingPos<ATT_NSB> sr;
      RingPos<PB> pr;
      RingPos<QB> qr;
      uint32_t wcnt = 0;
      bool ok = true;

      auto issue_pv = [&](int j) -> bool {
        if (j == 0 && !ptx::mbar_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x5500)) return false;
        const int vs = vr.idx, pb = pr.idx;
        if (!ptx::mbar_wait(&v_full[vs], vr.par, p.err, 0x5100 | vs)) return false;
        if (!ptx::mbar_wait(&p_full[pb], pr.par, p.err, 0x5200 | pb)) return false;
        ptx::tc_fence_after();
        if (issue) {
          const uint64_t pd = pd0 + (uint32_t)((pb * Cfg::P_TILE) >> 4), vd = vd0 + (uint32_t)((vs * Cfg::TILE) >> 4);
#pragma unroll
          for (int k = 0; k < ATT_BN / 16; ++k)    // 16 keys per MMA: 2 eight-key groups of V, 32 bytes of a P row
            ptx::umma_f16(tmem_base + Cfg::O_COL, pd + (uint32_t)(((k >> 2) * Cfg::SUB + (k & 3) * 32) >> 4),
                          vd + (uint32_t)((k * 2048) >> 4), p.idesc_pv, (j | k) != 0);
          ptx::umma_commit(&v_empty[vs]);
          ptx::umma_commit(&p_empty[pb]);
        }
        vr.advance(1); pr.advance(1);
        return true;
      };

      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int qt, h, b, klen; attn_tile(p, t, qt, h, b);
        const int nkv = attn_nkv(p, qt, b, klen);
        if (nkv == 0) continue;
        const int qb = qr.idx;
        if (!ptx::mbar_wait(&q_full[qb], qr.par, p.err, 0x5000 | qb)) { ok = false; break; }
        const uint64_t qd = qd0 + (uint32_t)((qb * Cfg::TILE) >> 4);
        for (int i = 0; i < 2 * nkv && ok; ++i) {
          const int ks = kr.idx, sb = sr.idx;
          if (!ptx::mbar_wait(&k_full[ks], kr.par, p.err, 0x5300 | ks)) { ok = false; break; }
          if (!ptx::mbar_wait(&s_empty[sb], sr.par ^ 1, p.err, 0x5400 | sb)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint64_t kd = kd0 + (uint32_t)((ks * Cfg::TILE) >> 4);
#pragma unroll
            for (int k = 0; k < DH / 16; ++k) {
              const uint32_t o = (uint32_t)(((k >> 2) * Cfg::SUB + (k & 3) * 32) >> 4);
              ptx::umma_f16(tmem_base + sb * ATT_BN, qd + o, kd + o, p.idesc_qk, k != 0);
            }
            ptx::umma_commit(&k_empty[ks]);
            ptx::umma_commit(&s_full[sb]);
            if (i == 2 * nkv - 1) ptx::umma_commit(&q_empty[qb]);
          }
          kr.advance(1); sr.advance(1);
          if (i >= nkv + 1) ok = issue_pv(i - nkv - 1);
        }
        if (ok) ok = issue_pv(nkv - 1);
        if (ok && issue) ptx::umma_commit(o_full);
        qr.advance(1);
        ++wcnt;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    const int quarter = warp & 3, cq = warp >> 2;
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;                                   // log2(e) / sqrt(dh)
    uint32_t scnt = 0, pcnt = 0, wcnt = 0;
    bool ok = true;

    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      int qt, h, b, klen; attn_tile(p, t, qt, h, b);
      const int nkv = attn_nkv(p, qt, b, klen);
      const int q0 = qt * ATT_BM, row_base = b * p.S, col0 = h * DH;
      const int q = q0 + r_loc;
      const bool row_ok = q < p.S;
      int kmax = klen - 1;
      if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);

      float m = -INFINITY;
      // ---- sweep 1: running row max (log2 domain)
      for (int i = 0; i < nkv; ++i, ++scnt) {
        const int sb = scnt % ATT_NSB;
        if (ok && !ptx::mbar_wait(&s_full[sb], (scnt / ATT_NSB) & 1, p.err, 0x6000 | sb)) ok = false;
        ptx::tc_fence_after();
        {
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + cq * 32, r);
          ptx::tmem_ld_wait();
          const int kb = i * ATT_BN + cq * 32;
          const int nvalid = min(32, kmax - kb + 1);
          if (__all_sync(0xffffffffu, nvalid >= 32)) {
            // every key of the piece allowed for every row of the warp: no per-element tests
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              mx0 = ptx::max3(mx0, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
              mx1 = ptx::max3(mx1, __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
            }
            m = fmaxf(m, fmaxf(mx0, mx1) * c2);
          } else if (nvalid > 0) {
            float smax = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) smax = fmaxf(smax, j < nvalid ? __uint_as_float(r[j]) : -INFINITY);
            m = fmaxf(m, smax * c2);
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_empty[sb]);
      }
      float2* st = stats + (wcnt & 1) * 4 * ATT_BM;
      st[cq * ATT_BM + r_loc] = make_float2(m, 0.f);
      asm volatile("bar.sync 1, 512;" ::: "memory");
      {
        float mf = -INFINITY;
#pragma unroll
        for (int g = 0; g < 4; ++g) mf = fmaxf(mf, st[g * ATT_BM + r_loc].x);
        m = mf;
      }
      const float mneg = m > -INFINITY ? -m : 0.f;            // a row without keys: every e is masked to 0 below

      // ---- sweep 2: e = 2^(t - m) <= 1 as FP16 / BF16 into shared memory (two 64-key sub-tiles, 128-byte swizzle) and the
      // row sum of the e in FP32; the sum is divided out of the accumulator in the epilogue (one exponential per score:
      // the first sweep needs the maximum only)
      float l2a = 0.f, l2b = 0.f;
      for (int j = 0; j < nkv; ++j, ++scnt, ++pcnt) {
        const int sb = scnt % ATT_NSB, pb = pcnt % PB;
        if (ok && !ptx::mbar_wait(&s_full[sb], (scnt / ATT_NSB) & 1, p.err, 0x6100 | sb)) ok = false;
        if (ok && !ptx::mbar_wait(&p_empty[pb], ((pcnt / PB) & 1) ^ 1, p.err, 0x6200 | pb)) ok = false;
        ptx::tc_fence_after();
        {
          const uint32_t prow = ptx::smem_u32(sP + pb * Cfg::P_TILE) + (cq >> 1) * Cfg::SUB + (r_loc >> 3) * 1024 + (r_loc & 7) * 128;
          uint32_t r[32];
          ptx::tmem_ld32(t_lane + sb * ATT_BN + cq * 32, r);
          ptx::tmem_ld_wait();
          const int kb = j * ATT_BN + cq * 32;
          const int nvalid = min(32, kmax - kb + 1);
          uint32_t w[16];
          if (__all_sync(0xffffffffu, nvalid >= 32)) {
            const float2 c22 = make_float2(c2, c2), nm2 = make_float2(mneg, mneg);
            float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float2 tt = __ffma2_rn(make_float2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), c22, nm2);
              const float2 ev = make_float2(ex2f(tt.x), ex2f(tt.y));
              acc2 = __fadd2_rn(acc2, ev);
              w[e] = fp2(ev.x, ev.y, in_dt);
            }
            l2a += acc2.x; l2b += acc2.y;
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              float a = ex2f(fmaf(__uint_as_float(r[2 * e]), c2, mneg));
              float c = ex2f(fmaf(__uint_as_float(r[2 * e + 1]), c2, mneg));
              if (2 * e >= nvalid) a = 0.f;
              if (2 * e + 1 >= nvalid) c = 0.f;
              l2a += a; l2b += c;
              w[e] = fp2(a, c, in_dt);
            }
          }
          const int c16 = (cq & 1) * 4;                      // first 16-byte chunk of this thread's 64 bytes
#pragma unroll
          for (int g = 0; g < 4; ++g)
            st_shared16(prow + (((c16 + g) ^ (r_loc & 7)) << 4), w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) { ptx::mbar_arrive(&s_empty[sb]); ptx::mbar_arrive(&p_full[pb]); }
      }

      // ---- the row sum from the four column parts; max P = 1 / l for the calibration observer (Eq. 16)
      st[cq * ATT_BM + r_loc].y = l2a + l2b;
      asm volatile("bar.sync 1, 512;" ::: "memory");
      const float l = (st[r_loc].y + st[ATT_BM + r_loc].y) + (st[2 * ATT_BM + r_loc].y + st[3 * ATT_BM + r_loc].y);
      const float inv_l = l > 0.f ? 1.0f / l : 0.f;
      if (p.p_absmax != nullptr && cq == 0) {
        float pm = row_ok ? inv_l : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) pm = fmaxf(pm, __shfl_xor_sync(0xffffffffu, pm, o));
        if (lane == 0 && pm > 0.f) atomicMax(reinterpret_cast<unsigned int*>(p.p_absmax), __float_as_uint(pm));
      }

      // ---- epilogue
      uint32_t r[32];
      if (nkv > 0) {
        if (ok && !ptx::mbar_wait(o_full, wcnt & 1, p.err, 0x6300)) ok = false;
        ptx::tc_fence_after();
        if (cq * 32 < DH) {
          ptx::tmem_ld32(t_lane + Cfg::O_COL + cq * 32, r);
          ptx::tmem_ld_wait();
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(o_empty);
        ++wcnt;
      }
      if (nkv == 0) {
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = 0;
      } else if (cq * 32 < DH) {
        // the accumulator holds sum_k e V: the row sum is divided out here
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * inv_l);
      }
      if (p.obs_col != nullptr && cq * 32 < DH) {
        // calibration observer: per-column maximum over the tile's 32 rows of this warp, rounded as the store rounds
        // (rounding is monotonic and symmetric, so the maximum of the rounded values is the rounded maximum)
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const uint32_t mx = __reduce_max_sync(0xffffffffu, row_ok ? (r[j] & 0x7fffffffu) : 0u);
          if (lane == j) mine = mx;
        }
        const uint32_t h = fp2(__uint_as_float(mine), 0.f, p.out_dt) & 0xffffu;
        const float stored = p.out_dt == HERO_F16 ? __half2float(__ushort_as_half((unsigned short)h)) : __uint_as_float(h << 16);
        if (stored > 0.f) atomicMax(reinterpret_cast<int*>(p.obs_col) + col0 + cq * 32 + lane, __float_as_int(stored));
      }
      if (cq * 32 < DH && row_ok) {
        const long long grow = (long long)(row_base + q);
        const int gcol = col0 + cq * 32;
        if (p.out_dt == HERO_I8) {
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) / __ldg(p.out_scale + (gcol + j) * p.out_scale_stride);
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
          for (int g = 0; g < 4; ++g)
            st_g16(dst + 8 * g, fp2(__uint_as_float(r[8 * g]), __uint_as_float(r[8 * g + 1]), p.out_dt),
                   fp2(__uint_as_float(r[8 * g + 2]), __uint_as_float(r[8 * g + 3]), p.out_dt),
                   fp2(__uint_as_float(r[8 * g + 4]), __uint_as_float(r[8 * g + 5]), p.out_dt),
                   fp2(__uint_as_float(r[8 * g + 6]), __uint_as_float(r[8 * g + 7]), p.out_dt));
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == ATT_MMA_WARP) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int DH>
static hero_status launch_attn_fp(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = AttnFpCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  const bool bf = a->dtype == HERO_BF16;
  CUtensorMap tq, tk, tv;
  hero_status st;
  // every load is one [128 rows x 64 elements] sub-tile: 128-byte rows, 128-byte swizzle
  if ((st = make_tmap_2d(h, &tq, a->q, 2, !bf, bf, rows, cols, (uint64_t)a->ld * 2, 64, ATT_BM, 128)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 2, !bf, bf, rows, cols, (uint64_t)a->ld * 2, 64, ATT_BN, 128)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 2, !bf, bf, rows, cols, (uint64_t)a->ld * 2, 64, ATT_BN, 128)) != HERO_OK) return st;
  const uint32_t fmt = bf ? 1 : 0;
  p.idesc_qk = ptx::make_idesc(1, fmt, fmt, 0, 0, ATT_BM, ATT_BN);   // F32 accumulate, both operands K-major
  p.idesc_pv = ptx::make_idesc(1, fmt, fmt, 0, 1, ATT_BM, DH);       // V is MN-major
  auto kern = attn_fp_kernel<DH>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  const long long tiles = (long long)p.nqt * a->nh * a->B;
  const int grid = (int)(tiles < h->sm_count ? tiles : h->sm_count);
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(ATT_THREADS), Cfg::SMEM_BYTES, stream, tq, tk, tv, p, a->dtype));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

hero_status attn_fp_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  p.c2 = (float)(1.4426950408889634 / sqrt((double)a->dh));
  if (a->dh == 64) return launch_attn_fp<64>(h, a, p, stream);
  return launch_attn_fp<128>(h, a, p, stream);
}

}  // namespace hero
