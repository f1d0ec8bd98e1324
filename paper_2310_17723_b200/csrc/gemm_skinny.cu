// GeMM^quant for few rows (M <= 128: the decode step of a generative model, or a short batch): the same operation
// and epilogue as gemm.cu (Sec. 2.2.2 Eq. 14, 18, 20-23; Sec. 2.2.3 Eq. 28-30, 32), organised for what bounds it here,
// which is streaming the weight matrix out of HBM once.
//
// The roles of the operands are swapped on the tensor core: a CTA takes 128 output features (rows of W [N][K]) as the
// UMMA M dimension and the MT >= M activation rows as its N dimension, so the accumulator D^T [128 features][MT rows]
// needs MT tensor-memory columns and no tensor-core work is spent on padding rows.  To put every SM to work on one
// weight matrix the K dimension is split over a thread-block cluster of CS <= 8 CTAs; each keeps its partial sums on
// chip, the CTAs exchange them through distributed shared memory (INT32 sums are exact in any order; FP32 sums are
// added in rank order, so the result does not depend on timing) and each CTA finishes 128 / CS features: scales, bias,
// activation, requantization, store.  No workspace in global memory, no atomics, no second launch.
//
//   warps 0-3  wait for the accumulator, move it to shared memory, reduce across the cluster, epilogue
//   warp  4    TMA producer: W tile [128 x 128 B] and activation tile [MT x 128 B] per K step, 128-byte swizzled
//   warp  5    UMMA issuer and owner of the tensor-memory allocation
// Every barrier wait is bounded; on expiry the CTA records a code, skips its stores and still joins the cluster barriers.
#include "gemm_common.cuh"

namespace hero {

constexpr int SK_THREADS = 192;
constexpr int SK_TMA_WARP = 4, SK_MMA_WARP = 5;
constexpr int SK_BN = 128;                 // output features per CTA

template <int MT>
struct SkinnyCfg {
  static constexpr int W_BYTES = SK_BN * GEMM_BK_BYTES;
  static constexpr int X_BYTES = MT * GEMM_BK_BYTES;
  static constexpr int STAGE_BYTES = W_BYTES + X_BYTES;
  static constexpr int STAGES = MT <= 16 ? 6 : (MT <= 32 ? 5 : (MT <= 64 ? 4 : 3));   // about 100 KB: two CTAs per SM
  static constexpr int PARTIAL_BYTES = MT * SK_BN * 4;                                // aliases the drained stages
  static constexpr int TMEM_COLS = MT < 32 ? 32 : MT;
  static constexpr int SMEM_BYTES = 1024 /*align slack*/ + STAGES * STAGE_BYTES + 256 /*barriers*/;
  static_assert(PARTIAL_BYTES <= STAGES * STAGE_BYTES, "partial sums must fit in the stage buffers");
};

// (not volatile, no memory clobber: the reads of several rows may be in flight together; every address derives from a
// mapa issued after the cluster barrier, which keeps them behind it)
__device__ __forceinline__ uint32_t ld_shared_cluster(uint32_t cluster_addr) {
  uint32_t v;
  asm("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr));
  return v;
}

// One output element: v = acc * rs * cs + bias; a = act(v) * post; INT8: clip(Round(a)) | e4m3 | F16 / BF16 | raw INT32.
// The arithmetic follows the wide kernels' epilogue step for step (the output factor is folded into cs and bias when
// there is no activation), so both give the same bits for the same accumulator.
template <bool INT8>
__device__ __forceinline__ void skinny_store(const GemmParams& p, int act, uint32_t acc_bits, int m, int n, float rs, float cs,
                                             float bias, float post) {
  const long long at = (long long)m * p.out_ld + n;
  if (p.out_dt == HERO_I32) {
    reinterpret_cast<int*>(p.out)[at] = (int)acc_bits;
    return;
  }
  const float acc = INT8 ? (float)(int)acc_bits : __uint_as_float(acc_bits);
  float y;
  if (act == HERO_ACT_NONE) {
    y = fmaf(acc * rs, cs * post, bias * post);
  } else {
    const float x = fmaf(acc * rs, cs, bias);
    y = (act == HERO_ACT_GELU_ERF ? gelu_erf_f(x) : gelu_tanh_f(x)) * post;
  }
  if (p.out_dt == HERO_I8) {
    const float r = fminf(fmaxf(y + ROUND_MAGIC, ROUND_MAGIC - 127.0f), ROUND_MAGIC + 127.0f);   // RNE in the adder, then clip
    reinterpret_cast<int8_t*>(p.out)[at] = (int8_t)(__float_as_uint(r) & 0xff);
  } else if (p.out_dt == HERO_F8) {
    reinterpret_cast<uint8_t*>(p.out)[at] = (uint8_t)(ptx::f32x2_to_e4m3x2(y, 0.0f) & 0xff);
  } else if (p.out_dt == HERO_F16) {
    reinterpret_cast<__half*>(p.out)[at] = __float2half_rn(y);
  } else {
    reinterpret_cast<__nv_bfloat16*>(p.out)[at] = __float2bfloat16_rn(y);
  }
}

template <int MT, bool INT8>
__global__ void __launch_bounds__(SK_THREADS) gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmW,
                                                                 const __grid_constant__ CUtensorMap tmX,
                                                                 const GemmParams p, const int act) {
  using Cfg = SkinnyCfg<MT>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * Cfg::STAGE_BYTES);
  uint64_t* full = bars;                    // [STAGES] TMA -> MMA
  uint64_t* empty = bars + STAGES;          // [STAGES] MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;   // MMA -> epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  uint32_t* partial = reinterpret_cast<uint32_t*>(tiles);   // [MT][128], written once the stages are drained

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cs_n = gridDim.x;               // cluster size = K splits (the cluster spans the grid's x dimension)
  const int rank = (int)ptx::cluster_ctarank();
  const int n0 = blockIdx.y * SK_BN;
  const int kb0 = (int)((long long)p.num_kb * rank / cs_n), kb1 = (int)((long long)p.num_kb * (rank + 1) / cs_n);

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&full[i], 1); ptx::mbar_init(&empty[i], 1); }
    ptx::mbar_init(acc_full, 1);
    ptx::fence_mbar_init();
  }
  if (warp == SK_MMA_WARP) {
    ptx::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  if (warp == SK_TMA_WARP && lane == 0) { ptx::prefetch_tmap(&tmW); ptx::prefetch_tmap(&tmX); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch_dependents();

  bool have_acc = false;                    // epilogue warps: this CTA's partial sums reached shared memory
  if (warp == SK_TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer
    // (this loop and the issuer's: whole warp, one elected lane issues; uniform control flow keeps the addresses in the
    // uniform datapath and the serial chains short)
    {
      const bool issue = ptx::elect_one();
      const int kelems = GEMM_BK_BYTES / p.elem_bytes;
      int stage = 0; uint32_t phase = 0;
      // The weights do not depend on the previous kernel of the stream: their first tiles are requested before the
      // dependency wait, the activation tiles after it (both complete the same barrier).
      const int pre = min(kb1 - kb0, STAGES);
      if (issue) {
        for (int i = 0; i < pre; ++i) {
          ptx::mbar_expect_tx(&full[i], Cfg::STAGE_BYTES);
          ptx::tma_load_2d(tiles + i * Cfg::STAGE_BYTES, &tmW, (kb0 + i) * kelems, n0, &full[i]);
        }
      }
      ptx::pdl_wait();
      for (int kb = kb0; kb < kb1; ++kb) {
        uint8_t* w_dst = tiles + stage * Cfg::STAGE_BYTES;
        const bool late = kb - kb0 >= pre;
        if (late && !ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x900 | stage)) break;
        if (issue) {
          if (late) {
            ptx::mbar_expect_tx(&full[stage], Cfg::STAGE_BYTES);
            ptx::tma_load_2d(w_dst, &tmW, kb * kelems, n0, &full[stage]);
          }
          ptx::tma_load_2d(w_dst + Cfg::W_BYTES, &tmX, kb * kelems, 0, &full[stage]);
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      // drain: every copy this thread started has been consumed before the stages are reused or the CTA exits
      for (int i = 0; i < STAGES; ++i) {
        if (!ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x980 | stage)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == SK_MMA_WARP) {
    // ------------------------------------------------------------------ UMMA issuer
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t desc_base = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);
      const uint64_t ad0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles));
      const uint64_t bd0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles) + Cfg::W_BYTES);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(&full[stage], phase, p.err, 0xA00 | stage)) { ok = false; break; }
        ptx::tc_fence_after();
        if (issue) {
          const uint32_t so = (uint32_t)(stage * Cfg::STAGE_BYTES) >> 4;
#pragma unroll
          for (int k = 0; k < GEMM_BK_BYTES / 32; ++k) {
            const uint64_t ad = ad0 + (so + 2 * k), bd = bd0 + (so + 2 * k);
            const uint32_t accumulate = (kb != kb0 || k != 0) ? 1u : 0u;
            if constexpr (INT8) ptx::umma_i8(tmem_base, ad, bd, p.idesc, accumulate);
            else if (p.f8) ptx::umma_f8(tmem_base, ad, bd, p.idesc, accumulate);
            else ptx::umma_f16(tmem_base, ad, bd, p.idesc, accumulate);
          }
          ptx::umma_commit(&empty[stage]);
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      if (ok && issue) ptx::umma_commit(acc_full);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ accumulator -> shared memory (feature-minor)
    ptx::pdl_wait();                                        // before this warp's first global access
    have_acc = __all_sync(0xffffffffu, ptx::mbar_wait(acc_full, 0, p.err, 0xB00));
    if (have_acc) {
      ptx::tc_fence_after();
      const int nl = warp * 32 + lane;                      // TMEM lane = feature within the tile
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll
      for (int c = 0; c < MT; c += 16) {
        uint32_t r[16];
        ptx::tmem_ld16(taddr + c, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) partial[(c + j) * SK_BN + nl] = r[j];
      }
    }
  }

  // ---- the partial sums of all K splits are in place
  ptx::tc_fence_before();
  ptx::cluster_sync();
  if (warp < 4 && have_acc) {
    const int R = SK_BN / cs_n;                             // features this CTA finishes
    const int tid = threadIdx.x;                            // 0..127
    const uint32_t base = ptx::smem_u32(partial);
    const int rows = min(p.M, MT);
    // R divides 128, so a thread keeps one feature n and walks the rows m = tid / R, tid / R + 128 / R, ...
    const int nl = rank * R + tid % R, n = n0 + nl;
    const bool n_ok = n < p.N;
    const float cs = (n_ok && p.cs) ? __ldg(p.cs + n) : 1.0f, bias = (n_ok && p.bias) ? __ldg(p.bias + n) : 0.0f;
    const float post = (n_ok && p.post) ? __ldg(p.post + n) : 1.0f;
    uint32_t peer[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) peer[q] = ptx::mapa(base + (uint32_t)nl * 4u, q < cs_n ? q : 0);
#pragma unroll 4
    for (int m = tid / R; m < rows; m += 128 / R) {
      const uint32_t off = (uint32_t)(m * SK_BN) * 4u;
      uint32_t v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = q < cs_n ? ld_shared_cluster(peer[q] + off) : 0u;
      uint32_t acc_bits;
      if constexpr (INT8) {
        int acc = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) acc += (int)v[q];
        acc_bits = (uint32_t)acc;
      } else {
        float acc = __uint_as_float(v[0]);                   // rank order; absent ranks contribute +0
#pragma unroll
        for (int q = 1; q < 8; ++q) acc += __uint_as_float(v[q]);
        acc_bits = __float_as_uint(acc);
      }
      if (n_ok) skinny_store<INT8>(p, act, acc_bits, m, n, p.rs ? __ldg(p.rs + m) : 1.0f, cs, bias, post);
    }
  }
  // ---- nobody leaves while a peer may still read its shared memory
  ptx::cluster_sync();
  if (warp == SK_MMA_WARP) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int MT, bool INT8>
static hero_status launch_skinny(hero_handle* h, const CUtensorMap& tmW, const CUtensorMap& tmX, const GemmParams& p, int act,
                                 int splits, cudaStream_t stream) {
  using Cfg = SkinnyCfg<MT>;
  auto kern = gemm_skinny_kernel<MT, INT8>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)splits, (unsigned)p.num_n_tiles);
  cfg.blockDim = dim3(SK_THREADS);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)splits; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_take_fence(stream) ? 1 : 2;   // a fenced stream: ordinary serialisation
  {
    LaunchScope scope(h, stream, KERNEL_GEMM);
    HERO_CUDA(cudaLaunchKernelEx(&cfg, kern, tmW, tmX, p, act));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

// M <= 128 rows.  `p` arrives filled by hero_w8a8_linear (sizes, vectors, output, error word).
hero_status run_skinny(hero_handle* h, const hero_linear_args* a, GemmParams& p, cudaStream_t s) {
  const bool int8 = a->A.dtype == HERO_I8, f8 = a->A.dtype == HERO_F8, bf = a->A.dtype == HERO_BF16;
  const int eb = (int8 || f8) ? 1 : 2;
  const int kbox = GEMM_BK_BYTES / eb;
  const int mt = p.M <= 16 ? 16 : (p.M <= 32 ? 32 : (p.M <= 64 ? 64 : 128));
  p.num_n_tiles = (p.N + SK_BN - 1) / SK_BN;
  p.idesc = int8 ? ptx::make_idesc(2, 1, 1, 0, 0, SK_BN, mt)
                 : (f8 ? ptx::make_idesc(1, 0, 0, 0, 0, SK_BN, mt) : ptx::make_idesc(1, bf ? 1 : 0, bf ? 1 : 0, 0, 0, SK_BN, mt));
  // K splits: enough CTAs for two per SM, at most 8 (the portable cluster size), a power of two, at least one K step each
  int splits = 1;
  while (splits < 8 && splits * 2 <= p.num_kb && (long long)p.num_n_tiles * splits * 2 <= 2ll * h->sm_count + h->sm_count / 4) splits *= 2;
  CUtensorMap tmW, tmX;
  hero_status st = make_tmap_2d(h, &tmW, a->W, eb, a->A.dtype == HERO_F16, bf, (uint64_t)p.N, (uint64_t)p.K, (uint64_t)a->ldw * eb,
                                kbox, SK_BN, 128);
  if (st != HERO_OK) return st;
  st = make_tmap_2d(h, &tmX, a->A.data, eb, a->A.dtype == HERO_F16, bf, (uint64_t)p.M, (uint64_t)p.K, (uint64_t)a->A.ld * eb, kbox,
                    mt, 128);
  if (st != HERO_OK) return st;
  switch (mt) {
    case 16: return int8 ? launch_skinny<16, true>(h, tmW, tmX, p, a->act, splits, s) : launch_skinny<16, false>(h, tmW, tmX, p, a->act, splits, s);
    case 32: return int8 ? launch_skinny<32, true>(h, tmW, tmX, p, a->act, splits, s) : launch_skinny<32, false>(h, tmW, tmX, p, a->act, splits, s);
    case 64: return int8 ? launch_skinny<64, true>(h, tmW, tmX, p, a->act, splits, s) : launch_skinny<64, false>(h, tmW, tmX, p, a->act, splits, s);
    default: return int8 ? launch_skinny<128, true>(h, tmW, tmX, p, a->act, splits, s) : launch_skinny<128, false>(h, tmW, tmX, p, a->act, splits, s);
  }
}

}  // namespace hero
