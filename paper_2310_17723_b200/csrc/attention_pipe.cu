// INT8 attention core (Sec. 2.2.2 Eq. 15-17) for sequences of at most 512 keys, as a pipeline of specialised warps.
//
// The static scale s_p of Eq. 16 quantizes the fully normalised probability, so a row's maximum and sum must be
// known before any of its P codes can be formed.  The whole score row therefore stays in tensor memory between the two
// steps, and the two steps are given to DIFFERENT warps so that the exponentials of one tile (bound by the
// special-function unit) run beside the scaling, rounding and packing of the previous tile (FMA and byte-permute work):
//
//   warps 0-7   exponential warps: lane quarter w % 4; the group w / 4 takes every other 64-key score block of a tile.
//               Per block: e = 2^(t c2 - mp) with mp the running maximum of the thread's pieces so far, written back
//               over the scores (tcgen05.st); running (max, sum) in registers; mp per piece and the final (max, sum) go
//               to shared memory.  One exponential per score.
//   warps 8-15  pack warps: lane quarter w % 4, column half w / 4 of every block.  Combine the two halves' statistics, then per block
//               P_u8 = Round(e 2^(mp - m) / (l s_p)) (one FMA with the 1.5 * 2^23 constant, byte permutes) into the UMMA
//               operand tile in shared memory; afterwards the tile's output stage (Eq. 17) from the accumulator.
//   warp 16     TMA producer: Q tile, K tiles of 128 keys, V tiles of 64 keys in the order P V consumes them.
//   warp 17     Q K^T issuer (one lane): a block as soon as its tensor-memory columns are free, running ahead into the
//               next tile while the current one is packed.
//   warp 18     P V issuer (one lane): a block as soon as its P tile is full.
//
// Tensor memory (512 columns): a ring of 64-column score blocks (7 for dh = 64, 6 for dh = 128) followed by the output
// accumulator (dh columns).  A tile of up to 7 (6) blocks lives in the ring alone; the ring slots it does not use let the
// next tile's first blocks be computed before any of its own are released.  A tile of 8 blocks (512 keys, dh = 64) is one
// slot short: its last block is computed FIRST, its e values go to a stash in shared memory instead of back to tensor
// memory, and its slot is handed on at once, so the tile never holds more than the ring.  (Putting that block over the
// accumulator's columns instead would chain every tile behind the previous tile's output stage.)  dh = 128 with more
// than 384 keys is left to the kernel of attention_resident.cu.
#include "attention_common.cuh"

namespace hero {

constexpr int PB = 64;                 // keys per score block = tensor-memory columns per block
constexpr int PIPE_EXP_WARPS = 8, PIPE_PACK_WARPS = 8;
constexpr int PIPE_TMA_WARP = 16, PIPE_QK_WARP = 17, PIPE_PV_WARP = 18;
constexpr int PIPE_THREADS = 20 * 32;  // warp 19 idles: register reallocation works on whole groups of four warps
// Registers per thread after the reallocation at kernel entry: every warp starts at the launch-bound figure (96 at 640
// threads).  The helper group (TMA / issuers) gives most of its registers back and the exponential warps, which keep two
// score blocks in flight, take them.  An increase can only be served from what the CTA's own warps have released (it
// blocks until then, and for ever if that never suffices), so the books must balance:
//   8 x 32 x (120 - 96) = 6144 <= 4 x 32 x (96 - 40) = 7168.
constexpr int PIPE_REGS_EXP = 120, PIPE_REGS_HELPER = 40;
static_assert(PIPE_EXP_WARPS == PIPE_PACK_WARPS, "a ring slot is released by eight arrivals, from either group");
static_assert(PIPE_EXP_WARPS * (PIPE_REGS_EXP - 96) <= 4 * (96 - PIPE_REGS_HELPER),
              "register increases must be covered by the helper group's release");
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
constexpr int PIPE_NPB = 4;            // P operand tiles (128 x 64 bytes) in shared memory
constexpr int PIPE_MAXB = 8;           // score blocks of a tile at most (512 keys)


template <int DH>
struct PipeCfg {
  static constexpr int NRING = (512 - DH) / PB;          // ring blocks: 7 (dh 64) or 6 (dh 128)
  static constexpr bool STASH = NRING == PIPE_MAXB - 1;  // an 8-block tile passes its last block through shared memory
  static constexpr int O_COL = NRING * PB;
  static constexpr int Q_TILE = ATT_BM * DH;
  static constexpr int K_TILE = PB * DH;
  static constexpr int V_TILE = PB * DH;
  static constexpr int P_TILE = ATT_BM * PB;
  static constexpr int KST = 8;
  static constexpr int VST = 8;
  static constexpr int OFF_K = 2 * Q_TILE;
  static constexpr int OFF_V = OFF_K + KST * K_TILE;
  static constexpr int OFF_P = OFF_V + VST * V_TILE;
  static constexpr int OFF_PM = OFF_P + PIPE_NPB * P_TILE;                  // float [2][MAXB][2][128]: piece maxima
  static constexpr int OFF_ST = OFF_PM + 2 * PIPE_MAXB * 2 * ATT_BM * 4;     // float2 [2][2][128]: (max, sum) per half
  static constexpr int OFF_OSC = OFF_ST + 2 * 2 * ATT_BM * 8;                // float [8 pack warps][DH / 2]: output factors
  static constexpr int OFF_STASH = OFF_OSC + PIPE_PACK_WARPS * (DH / 2) * 4;  // float [2][64 columns][128 rows]: the stashed block's e
  static constexpr int OFF_BARS = OFF_STASH + (STASH ? 2 * PB * ATT_BM * 4 : 0);
  static constexpr int NBARS = 4 + 2 * KST + 2 * VST + 2 * PIPE_MAXB + 4 + 2 * PIPE_NPB + 2;
  static constexpr int SMEM_BYTES = 1024 + OFF_BARS + NBARS * 8 + 16;
  static constexpr uint32_t SWZ = (DH == 128) ? ptx::SWZ_128B : ptx::SWZ_64B;
  static constexpr uint32_t SBO = 8 * DH;
};

struct PipeTile { int qt, h, b, klen, nb; };

// The tiles blockIdx.x, blockIdx.x + gridDim.x, ... of the persistent walk, decoded without a division per tile: tile t
// is (query tile nqt - 1 - t / (B nh), head (t mod B nh) mod nh, batch (t mod B nh) / nh) (late query tiles first, as in
// attn_tile); the quotients and remainders advance by constants.
struct PipeWalk {
  int t, hi, r, h, b;
  int G, dhi, dr, dh, db, bh, nh, B;
  __device__ __forceinline__ PipeWalk(const AttnParams& p, int t0, int grid) {
    bh = p.B * p.nh; nh = p.nh; B = p.B; G = grid;
    t = t0; hi = t0 / bh; r = t0 - hi * bh; b = r / nh; h = r - b * nh;
    dhi = grid / bh; dr = grid - dhi * bh; db = dr / nh; dh = dr - db * nh;
  }
  __device__ __forceinline__ void next() {
    t += G; hi += dhi; r += dr; h += dh; b += db;
    if (h >= nh) { h -= nh; ++b; }
    if (r >= bh) { r -= bh; ++hi; b -= B; }
  }
  // false when every key of the tile is masked (no tensor work: the rows are zero)
  __device__ __forceinline__ bool tile(const AttnParams& p, PipeTile& g) const {
    g.qt = p.nqt - 1 - hi; g.h = h; g.b = b;
    g.klen = p.S;
    if (p.key_len) g.klen = min(p.S, max(0, p.key_len[b]));
    int kv_end = g.klen;
    if (p.mask == HERO_MASK_CAUSAL) kv_end = min(kv_end, g.qt * ATT_BM + ATT_BM);
    g.nb = (kv_end + PB - 1) / PB;
    return g.nb > 0;
  }
};

// A global load that stays where it is written: the compiler may otherwise sink a load to its first use, which here is a
// whole tile later, on the critical path.
__device__ __forceinline__ float ld_nc_here(const float* ptr) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(ptr));
  return v;
}

// Bounded wait (mbarrier.try_wait with a suspend-time hint inside a bounded loop).
__device__ __forceinline__ bool pipe_wait(uint64_t* bar, uint32_t parity, int* err, int code) {
  return ptx::mbar_wait(bar, parity, err, code);
}

// A barrier wait for a whole group of warps: ONE warp polls the mbarrier, the others block on a hardware named
// barrier until it has seen the phase complete.  Eight warps polling the same word would spend a third of the SM's issue
// slots on polling loops.  `id`: the group's named barrier (1 and 3: the two groups of exponential warps, 2: the pack warps); every warp
// of a group must make the same sequence of calls.
template <int THREADS>
__device__ __forceinline__ bool pipe_group_wait(bool leader, int id, uint64_t* bar, uint32_t parity, int* err, int code, bool ok) {
  if (leader && ok) ok = pipe_wait(bar, parity, err, code);
  asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(THREADS) : "memory");
  return ok;
}

// The k-th block in Q K^T / exponential order: a tile that stashes computes its last block first.  Pack / P V order is
// the natural one (the stashed block last).
__device__ __forceinline__ int pipe_qk_block(int nb, bool stash, int k) { return stash ? (k == 0 ? nb - 1 : k - 1) : k; }

// One 32-column piece of a score block: raw scores in r (INT32, or FP32 for the e4m3 kind) become e = 2^(t c2 - mn) with
// mn = max(running maximum, piece maximum); the running (m, l) are updated.  nvalid < 32: only the first nvalid keys
// are allowed (the rest become exactly 0).
template <bool F8, bool FULL>
__device__ __forceinline__ void pipe_exp_piece(uint32_t (&r)[32], int nvalid, float c2, float& m, float& l) {
  float pmx;
  if constexpr (F8) {
    float f0 = -INFINITY, f1 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      f0 = fmaxf(f0, (FULL || e < nvalid) ? __uint_as_float(r[e]) : -INFINITY);
      f1 = fmaxf(f1, (FULL || e + 1 < nvalid) ? __uint_as_float(r[e + 1]) : -INFINITY);
    }
    pmx = fmaxf(f0, f1) * c2;
  } else {
    int i0 = INT_MIN, i1 = INT_MIN;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
      i0 = max(i0, max((FULL || e < nvalid) ? (int)r[e] : INT_MIN, (FULL || e + 1 < nvalid) ? (int)r[e + 1] : INT_MIN));
      i1 = max(i1, max((FULL || e + 2 < nvalid) ? (int)r[e + 2] : INT_MIN, (FULL || e + 3 < nvalid) ? (int)r[e + 3] : INT_MIN));
    }
    pmx = (float)max(i0, i1) * c2;
  }
  const float mn = fmaxf(m, pmx);
  const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-mn, -mn);
  float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
  for (int e = 0; e < 32; e += 2) {
    const float2 f = F8 ? make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]))
                        : make_float2((float)(int)r[e], (float)(int)r[e + 1]);
    float2 tt = __ffma2_rn(f, c22, nm2);
    if constexpr (!FULL) {                                   // a masked key: 2^(-inf) = +0 exactly
      if (e >= nvalid) tt.x = -INFINITY;
      if (e + 1 >= nvalid) tt.y = -INFINITY;
    }
    const float2 ev = make_float2(ex2f(tt.x), ex2f(tt.y));
    acc2 = __fadd2_rn(acc2, ev);
    r[e] = __float_as_uint(ev.x); r[e + 1] = __float_as_uint(ev.y);
  }
  l = l * ex2f(m - mn) + (acc2.x + acc2.y);                  // m = -inf before the first piece: 2^(-inf) = 0
  m = mn;
}

// 32 values e (FP32 bits in r) times the factor f -> 32 P codes packed into w[8].
template <bool F8>
__device__ __forceinline__ void pipe_pack32(const uint32_t (&r)[32], float f, uint32_t (&w)[8]) {
  const float2 f2v = make_float2(f, f), rm2 = make_float2(ATT_MAGIC, ATT_MAGIC);
  if constexpr (F8) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int e = 4 * k;
      const float2 a = __fmul2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v);
      const float2 c = __fmul2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), f2v);
      w[k] = ptx::f32x4_to_e4m3x4(a.x, a.y, c.x, c.y);       // saturates at 448 (s_p = max P / 448)
    }
  } else if (f <= 255.25f) {
    // e <= 1 in every piece, so e f cannot round above 255: no clip needed
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int e = 4 * k;
      w[k] = low_bytes4_u(fmaf(__uint_as_float(r[e]), f, ATT_MAGIC), fmaf(__uint_as_float(r[e + 1]), f, ATT_MAGIC),
                          fmaf(__uint_as_float(r[e + 2]), f, ATT_MAGIC), fmaf(__uint_as_float(r[e + 3]), f, ATT_MAGIC));
    }
  } else {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int e = 4 * k;
      const float2 a = __ffma2_rn(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), f2v, rm2);
      const float2 c = __ffma2_rn(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), f2v, rm2);
      w[k] = low_bytes4_u(fminf(a.x, ATT_MAGIC + 255.0f), fminf(a.y, ATT_MAGIC + 255.0f),
                          fminf(c.x, ATT_MAGIC + 255.0f), fminf(c.y, ATT_MAGIC + 255.0f));
    }
  }
}

// ROWMAX: the long-sequence-robust P quantizer (not in the paper): P~_u8 = Round(255 * 2^(t - m_row)), the row sum l of the
// un-quantized exponentials divided out in the output stage.  F8: e4m3 Q, K, V and an e4m3 P (static quantizer only):
// kind::f8f6f4 products, FP32 scores and accumulator.  PROBE: the raw scores, the P codes and the raw accumulators are
// also written to global memory (verification only).
template <int DH, bool ROWMAX, bool F8, bool PROBE>
__global__ void __launch_bounds__(PIPE_THREADS, 1)
attn_int8_pipe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnParams p) {
  using Cfg = PipeCfg<DH>;
  constexpr int KST = Cfg::KST, VST = Cfg::VST, NRING = Cfg::NRING;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + Cfg::OFF_K;
  uint8_t* sV = smem + Cfg::OFF_V;
  uint8_t* sP = smem + Cfg::OFF_P;
  float* pm_s = reinterpret_cast<float*>(smem + Cfg::OFF_PM);
  float2* st_s = reinterpret_cast<float2*>(smem + Cfg::OFF_ST);
  float* osc_s = reinterpret_cast<float*>(smem + Cfg::OFF_OSC);
  float* stash_s = reinterpret_cast<float*>(smem + Cfg::OFF_STASH);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BARS);
  uint64_t* q_full = bars;                      // [2]
  uint64_t* q_empty = q_full + 2;               // [2]
  uint64_t* k_full = q_empty + 2;               // [KST]
  uint64_t* k_empty = k_full + KST;             // [KST]
  uint64_t* v_full = k_empty + KST;             // [VST]
  uint64_t* v_empty = v_full + VST;             // [VST]
  uint64_t* s_full = v_empty + VST;             // [MAXB]  ring slot written by Q K^T
  uint64_t* s_free = s_full + PIPE_MAXB;        // [MAXB]  ring slot read out by every pack warp (stashed block: every exponential warp)
  uint64_t* t_full = s_free + PIPE_MAXB;        // [2]     every exponential warp is through with the tile of this parity
  uint64_t* t_empty = t_full + 2;               // [2]     every pack warp has read that tile's statistics (and stash)
  uint64_t* p_full = t_empty + 2;               // [NPB]
  uint64_t* p_empty = p_full + PIPE_NPB;        // [NPB]
  uint64_t* o_full = p_empty + PIPE_NPB;        // [1]
  uint64_t* o_empty = o_full + 1;               // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_empty + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.nqt * p.nh * p.B;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&q_full[i], 1); ptx::mbar_init(&q_empty[i], 1); ptx::mbar_init(&t_full[i], PIPE_EXP_WARPS); ptx::mbar_init(&t_empty[i], PIPE_PACK_WARPS); }
    for (int i = 0; i < KST; ++i) { ptx::mbar_init(&k_full[i], 1); ptx::mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < VST; ++i) { ptx::mbar_init(&v_full[i], 1); ptx::mbar_init(&v_empty[i], 1); }
    for (int i = 0; i < PIPE_MAXB; ++i) { ptx::mbar_init(&s_full[i], 1); ptx::mbar_init(&s_free[i], PIPE_PACK_WARPS); }
    for (int i = 0; i < PIPE_NPB; ++i) { ptx::mbar_init(&p_full[i], PIPE_PACK_WARPS); ptx::mbar_init(&p_empty[i], 1); }
    ptx::mbar_init(o_full, 1); ptx::mbar_init(o_empty, PIPE_PACK_WARPS);
    ptx::fence_mbar_init();
  }
  if (warp == PIPE_QK_WARP) { ptx::tmem_alloc(tmem_slot, 512); ptx::tmem_relinquish(); }
  if (warp == PIPE_TMA_WARP && lane == 0) { ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch_dependents();
  ptx::pdl_wait();                                       // the previous kernel's outputs are complete and visible from here on

  if (warp >= PIPE_TMA_WARP) {
  reg_dec<PIPE_REGS_HELPER>();                             // the helper group (its fourth warp has no work)
  if (warp == PIPE_TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer
    // (The three helper loops are walked by the whole warp, one elected lane issuing: with uniform control flow the
    // addresses stay in the uniform datapath, and a helper's turn-around time is part of every hand-off.)
    {
      const bool issue = ptx::elect_one();
      uint32_t kcnt = 0, vcnt = 0, wcnt = 0;
      bool ok = true;
      for (PipeWalk w(p, blockIdx.x, gridDim.x); w.t < total_tiles && ok; w.next()) {
        PipeTile g;
        if (!w.tile(p, g)) continue;
        const int row_base = g.b * p.S, col0 = g.h * DH;
        const int qb = wcnt & 1;
        if (!pipe_wait(&q_empty[qb], ((wcnt >> 1) & 1) ^ 1, p.err, 0x7000 | qb)) { ok = false; break; }
        if (issue) {
          ptx::mbar_expect_tx(&q_full[qb], Cfg::Q_TILE);
          ptx::tma_load_2d(sQ + qb * Cfg::Q_TILE, &tmQ, col0, row_base + g.qt * ATT_BM, &q_full[qb]);
        }
        const bool stash = g.nb > NRING;
        for (int k = 0; k < g.nb && ok; ++k, ++kcnt) {       // K blocks of 64 keys in Q K^T order
          const int j = pipe_qk_block(g.nb, stash, k);
          const int ks = kcnt % KST;
          if (!pipe_wait(&k_empty[ks], ((kcnt / KST) & 1) ^ 1, p.err, 0x7100 | ks)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&k_full[ks], Cfg::K_TILE);
            ptx::tma_load_2d(sK + ks * Cfg::K_TILE, &tmK, col0, row_base + j * PB, &k_full[ks]);
          }
        }
        for (int j = 0; j < g.nb && ok; ++j, ++vcnt) {       // V blocks of 64 keys in P V order
          const int vs = vcnt % VST;
          if (!pipe_wait(&v_empty[vs], ((vcnt / VST) & 1) ^ 1, p.err, 0x7200 | vs)) { ok = false; break; }
          if (issue) {
            ptx::mbar_expect_tx(&v_full[vs], Cfg::V_TILE);
            ptx::tma_load_2d(sV + vs * Cfg::V_TILE, &tmV, col0, row_base + j * PB, &v_full[vs]);
          }
        }
        ++wcnt;
      }
    }
    __syncwarp();
  } else if (warp == PIPE_QK_WARP) {
    // ------------------------------------------------------------------ Q K^T issuer: block after block, tile after tile
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t kmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // Q, K: K-major rows of DH bytes
      // descriptors differ only in the start-address field (address >> 4): one base per operand, small additions later
      const uint64_t qd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sQ)), kd0 = ptx::smem_desc(kmaj, ptx::smem_u32(sK));
      uint32_t wcnt = 0, kcnt = 0;
      RingPos<NRING> ring;
      bool ok = true;
      for (PipeWalk w(p, blockIdx.x, gridDim.x); w.t < total_tiles && ok; w.next()) {
        PipeTile g;
        if (!w.tile(p, g)) continue;
        const int qb = wcnt & 1;
        if (!pipe_wait(&q_full[qb], (wcnt >> 1) & 1, p.err, 0x8000 | qb)) { ok = false; break; }
        const uint64_t qd = qd0 + (uint32_t)((qb * Cfg::Q_TILE) >> 4);
        for (int k = 0; k < g.nb && ok; ++k, ++kcnt, ring.advance(1)) {
          const int ks = kcnt % KST, blk = ring.idx;
          if (!pipe_wait(&k_full[ks], (kcnt / KST) & 1, p.err, 0x8100 | ks)) { ok = false; break; }
          // the ring slot: whoever read the block that was there (the pack warps, or the exponential warps for a block
          // that went to the stash) is through with it
          if (!pipe_wait(&s_free[blk], ring.par ^ 1, p.err, 0x8200 | blk)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint64_t kd = kd0 + (uint32_t)((ks * Cfg::K_TILE) >> 4);
#pragma unroll
            for (int kk = 0; kk < DH / 32; ++kk) {
              if constexpr (F8) ptx::umma_f8(tmem_base + blk * PB, qd + 2 * kk, kd + 2 * kk, p.idesc_qk, kk != 0);
              else ptx::umma_i8(tmem_base + blk * PB, qd + 2 * kk, kd + 2 * kk, p.idesc_qk, kk != 0);
            }
            ptx::umma_commit(&s_full[blk]);
            ptx::umma_commit(&k_empty[ks]);
          }
        }
        if (ok && issue) ptx::umma_commit(&q_empty[qb]);
        ++wcnt;
      }
    }
    __syncwarp();
  } else if (warp == PIPE_PV_WARP) {
    // ------------------------------------------------------------------ P V issuer
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t pmaj = ptx::smem_desc_base(16, 512, ptx::SWZ_64B);        // P: K-major rows of 64 bytes
      constexpr uint64_t vmaj = ptx::smem_desc_base(16, Cfg::SBO, Cfg::SWZ);       // V: MN-major, 8-key groups
      const uint64_t pd0 = ptx::smem_desc(pmaj, ptx::smem_u32(sP)), vd0 = ptx::smem_desc(vmaj, ptx::smem_u32(sV));
      uint32_t wcnt = 0, vcnt = 0, pcnt = 0;
      bool ok = true;
      for (PipeWalk w(p, blockIdx.x, gridDim.x); w.t < total_tiles && ok; w.next()) {
        PipeTile g;
        if (!w.tile(p, g)) continue;
        // the accumulator's columns are free: the previous tile's output has been read
        if (!pipe_wait(o_empty, (wcnt & 1) ^ 1, p.err, 0x8400)) { ok = false; break; }
        for (int i = 0; i < g.nb && ok; ++i, ++vcnt, ++pcnt) {
          const int pb = pcnt % PIPE_NPB, vs = vcnt % VST;
          if (!pipe_wait(&v_full[vs], (vcnt / VST) & 1, p.err, 0x8600 | vs)) { ok = false; break; }
          if (!pipe_wait(&p_full[pb], (pcnt / PIPE_NPB) & 1, p.err, 0x8700 | pb)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint64_t pd = pd0 + (uint32_t)((pb * Cfg::P_TILE) >> 4), vd = vd0 + (uint32_t)((vs * Cfg::V_TILE) >> 4);
#pragma unroll
            for (int k = 0; k < PB / 32; ++k) {
              if constexpr (F8) ptx::umma_f8(tmem_base + Cfg::O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (i | k) != 0);
              else ptx::umma_i8(tmem_base + Cfg::O_COL, pd + 2 * k, vd + (uint32_t)((k * 32 * DH) >> 4), p.idesc_pv, (i | k) != 0);
            }
            ptx::umma_commit(&v_empty[vs]);
            ptx::umma_commit(&p_empty[pb]);
          }
        }
        if (ok && issue) ptx::umma_commit(o_full);
        ++wcnt;
      }
    }
    __syncwarp();
  }
  } else if (warp < PIPE_EXP_WARPS) {
    // ------------------------------------------------------------------ exponential warps
    // Two groups of four warps (one warp per lane quarter each).  A group takes every other block of a tile, all 64
    // columns of it, so the two warps that share a scheduler are always one block apart: while one waits for its block,
    // loads it or stores it, the other one's exponentials keep the special-function unit busy.
    reg_inc<PIPE_REGS_EXP>();
    const int quarter = warp & 3, grp = warp >> 2;
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float c2 = p.c2;
    const bool leader = quarter == 0;
    const int bar_id = 1 + 2 * grp;
    uint32_t wcnt = 0;
    RingPos<NRING> ring;                                     // the ring slot of the tile's first block (Q K^T order)
    bool ok = true;
    for (PipeWalk w(p, blockIdx.x, gridDim.x); w.t < total_tiles; w.next()) {
      PipeTile g;
      if (!w.tile(p, g)) continue;
      const int q = g.qt * ATT_BM + r_loc;
      int kmax = g.klen - 1;
      if (p.mask == HERO_MASK_CAUSAL) kmax = min(kmax, q);
      const int par = wcnt & 1;
      const bool stash = g.nb > NRING;
      // the statistics (and stash) slots of this parity are free: the pack warps are through with the tile two back.
      // (With spare ring slots the exponential warps could otherwise run several tiles ahead of the pack warps.)
      ok = pipe_group_wait<128>(leader, bar_id, &t_empty[par], ((wcnt >> 1) & 1) ^ 1, p.err, 0x9400 | par, ok);
      float* pm_row = pm_s + (par * PIPE_MAXB) * 2 * ATT_BM + r_loc;
      const long long probe_row = ((long long)(g.b * p.nh + g.h) * p.S + q) * p.S;
      float m = -INFINITY, l = 0.f;
      auto probe_scores = [&](const uint32_t (&r)[32], int key0) {
        if constexpr (PROBE) {
          if (p.dbg_scores && q < p.S) {
#pragma unroll
            for (int e = 0; e < 32; ++e) if (key0 + e < p.S) p.dbg_scores[probe_row + key0 + e] = (int)r[e];
          }
        }
      };
      // k: position in Q K^T order; every block takes the next ring slot; this group's blocks are every other one
#pragma unroll 1
      for (int k = (grp ^ (int)wcnt) & 1; k < g.nb; k += 2) {
        const int j = pipe_qk_block(g.nb, stash, k);
        int blk;
        uint32_t blk_par;
        ring.at(k, blk, blk_par);
        ok = pipe_group_wait<128>(leader, bar_id, &s_full[blk], blk_par, p.err, 0x9000 | blk, ok);
        ptx::tc_fence_after();
        const int key0 = j * PB;
        const bool to_stash = stash && k == 0;
        float* stash_dst = stash_s + (par * PB) * ATT_BM + r_loc;
        {
          // one 32-column piece after the other, in a rolled loop: the kernel's five roles share the instruction caches, and
          // a block's 64 exponentials unrolled as one straight line (twice the code) ran slower than this, not faster
#pragma unroll 1
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t r[32];
            ptx::tmem_ld32(t_lane + blk * PB + hh * 32, r);
            ptx::tmem_ld_wait();
            probe_scores(r, key0 + hh * 32);
            const int nvalid = kmax - (key0 + hh * 32) + 1;
            if (__all_sync(0xffffffffu, nvalid >= 32)) {
              pipe_exp_piece<F8, true>(r, 32, c2, m, l);
            } else if (nvalid > 0) {
              pipe_exp_piece<F8, false>(r, nvalid, c2, m, l);
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) r[e] = 0;           // every key of the piece masked
            }
            if (Cfg::STASH && to_stash) {
#pragma unroll
              for (int e = 0; e < 32; ++e) stash_dst[(hh * 32 + e) * ATT_BM] = __uint_as_float(r[e]);
            } else {
              ptx::tmem_st32(t_lane + blk * PB + hh * 32, r);
            }
            pm_row[(j * 2 + hh) * ATT_BM] = m;
          }
          if (Cfg::STASH && to_stash) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) { ptx::mbar_arrive(&s_free[blk]); ptx::mbar_arrive(&s_free[blk]); }
          }
        }
      }
      ptx::tmem_st_wait();
      st_s[(par * 2 + grp) * ATT_BM + r_loc] = make_float2(m, l);   // this group's blocks: their running maximum and sum
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&t_full[par]);
      ring.advance(g.nb);
      ++wcnt;
    }
  } else {
    // ------------------------------------------------------------------ pack + output warps
    const int quarter = warp & 3, half = (warp >> 2) & 1;
    const int r_loc = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    constexpr int OW = DH / 2;                               // output columns of this warp: half * OW .. + OW - 1
    float* osc = osc_s + (warp - PIPE_EXP_WARPS) * OW;
    uint32_t wcnt = 0, pcnt = 0;
    RingPos<NRING> ring;                                     // the ring slot of the tile's first block (Q K^T order)
    bool ok = true;
    // the per-column output scales of a tile are fetched one tile ahead (a global load in front of every tile would
    // stand on the pack warps' critical path)
    PipeTile g, gn;
    bool work = false, work_n = false;
    float osc_raw[OW / 32], osc_raw_n[OW / 32];
    auto fetch = [&](const PipeWalk& ww, PipeTile& gg, bool& wk, float (&raw)[OW / 32]) {
      if (ww.t >= total_tiles) return;
      wk = ww.tile(p, gg);
#pragma unroll
      for (int c = 0; c < OW / 32; ++c)
        raw[c] = is_q8(p.out_dt) ? ld_nc_here(p.out_scale + (long long)(gg.h * DH + half * OW + c * 32 + lane) * p.out_scale_stride) : 1.f;
    };
    PipeWalk w(p, blockIdx.x, gridDim.x);
    fetch(w, gn, work_n, osc_raw_n);
    for (; w.t < total_tiles;) {
      g = gn; work = work_n;
#pragma unroll
      for (int c = 0; c < OW / 32; ++c) osc_raw[c] = osc_raw_n[c];
      w.next();
      fetch(w, gn, work_n, osc_raw_n);
      const int q = g.qt * ATT_BM + r_loc;
      const bool row_ok = q < p.S;
      const long long grow = (long long)g.b * p.S + q;
      const int col0 = g.h * DH + half * OW;
      if (!work) {
        // every key masked: the rows are zero, no tensor work
        if (row_ok) {
          const int es = is_q8(p.out_dt) ? 1 : 2;
          uint8_t* dst = reinterpret_cast<uint8_t*>(p.out) + (grow * p.out_ld + col0) * es;
          for (int c = 0; c < OW * es / 16; ++c) st_g16(dst + 16 * c, 0u, 0u, 0u, 0u);
        }
        continue;
      }
      // this warp's per-column output factors s_p s_v / S_attn[j] (s_p s_v alone for an FP output)
      __syncwarp();
#pragma unroll
      for (int c = 0; c < OW / 32; ++c) osc[c * 32 + lane] = is_q8(p.out_dt) ? __fdividef(p.pv_scale, osc_raw[c]) : p.pv_scale;
      const int par = wcnt & 1;
      const bool stash = g.nb > NRING;
      const long long probe_row = ((long long)(g.b * p.nh + g.h) * p.S + q) * p.S;
      ok = pipe_group_wait<256>(warp == PIPE_EXP_WARPS, 2, &t_full[par], (wcnt >> 1) & 1, p.err, 0x9100 | par, ok);
      ptx::tc_fence_after();
      // ---- the row's maximum and sum from the two column halves
      const float2 sa = st_s[(par * 2 + 0) * ATT_BM + r_loc], sb = st_s[(par * 2 + 1) * ATT_BM + r_loc];
      const float m = fmaxf(sa.x, sb.x);
      float lsum = 0.f;
      if (m > -INFINITY) {
        if (sa.x > -INFINITY) lsum += sa.y * ex2f(sa.x - m);
        if (sb.x > -INFINITY) lsum += sb.y * ex2f(sb.x - m);
      }
      // static: P = e 2^(mp - m) / (l s_p); row-max: P~ = 255 e 2^(mp - m), the sum divided out in the output stage
      const float pscale = lsum > 0.f ? (ROWMAX ? 255.0f : __fdividef(p.inv_sp, lsum)) : 0.f;
      const float rowf = ROWMAX ? (lsum > 0.f ? 1.0f / lsum : 0.f) : 1.0f;
      const float* pm_row = pm_s + ((par * PIPE_MAXB) * 2 + half) * ATT_BM + r_loc;
      const int sw = (r_loc >> 1) & 3;
      // UMMA K-major operand tile with 64-byte rows and the 64-byte swizzle: 16-byte chunk c of row r sits at chunk
      // c ^ ((r >> 1) & 3) of the row; this warp owns chunks 2 half and 2 half + 1
      const uint32_t prow_off = r_loc * 64;
      const uint32_t ch0 = ((2 * half) ^ sw) << 4, ch1 = ((2 * half + 1) ^ sw) << 4;
      auto factor = [&](int j) { const float mp = pm_row[j * 2 * ATT_BM]; return mp > -INFINITY ? ex2f(mp - m) * pscale : 0.f; };
      auto probe_codes = [&](const uint32_t (&wd)[8], int j) {
        if constexpr (PROBE) {
          if (p.dbg_p && row_ok) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (j * PB + half * 32 + e < p.S) p.dbg_p[probe_row + j * PB + half * 32 + e] = (uint8_t)(wd[e >> 2] >> (8 * (e & 3)));
          }
        }
      };
      // One block per round, in key order: a P tile goes to the P V issuer, and its columns back to the Q K^T issuer, as
      // early as possible (the hand-offs between the roles, not the arithmetic, are what a tile's time is made of).
#pragma unroll 1
      for (int j = 0; j < g.nb; ++j) {
        const bool from_stash = stash && j == g.nb - 1;      // the block that was computed first and parked in shared memory
        int blk;
        uint32_t blk_par;
        ring.at(stash ? j + 1 : j, blk, blk_par);
        const int pb = pcnt % PIPE_NPB;
        uint32_t r[32];
        if (Cfg::STASH && from_stash) {
          const float* src = stash_s + (par * PB + half * 32) * ATT_BM + r_loc;
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(src[e * ATT_BM]);
        } else {
          ptx::tmem_ld32(t_lane + blk * PB + half * 32, r);
        }
        const float f = factor(j);
        if (!(Cfg::STASH && from_stash)) {
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&s_free[blk]);     // the block's columns may take the next tile's scores
        }
        ok = pipe_group_wait<256>(warp == PIPE_EXP_WARPS, 2, &p_empty[pb], ((pcnt / PIPE_NPB) & 1) ^ 1, p.err, 0x9200 | pb, ok);
        uint32_t wd[8];
        pipe_pack32<F8>(r, f, wd);
        probe_codes(wd, j);
        const uint32_t pr = ptx::smem_u32(sP + pb * Cfg::P_TILE) + prow_off;
        st_shared16(pr + ch0, wd[0], wd[1], wd[2], wd[3]);
        st_shared16(pr + ch1, wd[4], wd[5], wd[6], wd[7]);
        ptx::fence_proxy_async_smem();                       // generic-proxy writes -> visible to the UMMA (async proxy)
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[pb]);
        ++pcnt;
      }
      ring.advance(g.nb);
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&t_empty[par]);        // statistics and stash of this parity may be overwritten
      // ---- output stage (Eq. 17): X_attn = acc * s_p s_v (/ S_attn[j] -> Round -> INT8); OW columns per warp
      ok = pipe_group_wait<256>(warp == PIPE_EXP_WARPS, 2, o_full, wcnt & 1, p.err, 0x9300, ok);
      ptx::tc_fence_after();
      // 16 columns at a time in a rolled loop (this stage runs once per tile: its code should be small, not fast)
#pragma unroll 1
      for (int c0 = 0; c0 < OW; c0 += 16) {
        uint32_t r[16];
        ptx::tmem_ld16(t_lane + Cfg::O_COL + half * OW + c0, r);
        ptx::tmem_ld_wait();
        if (c0 + 16 >= OW) {                                 // the accumulator is in registers: the next tile may use its columns
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(o_empty);
        }
        if (row_ok) {
          const int gcol = col0 + c0;
          if constexpr (PROBE) {
            if (p.dbg_acc) {
              int* dst = p.dbg_acc + grow * ((long long)p.nh * p.dh) + gcol;
#pragma unroll
              for (int c = 0; c < 16; ++c) dst[c] = (int)r[c];
            }
          }
          const float4* o4 = reinterpret_cast<const float4*>(osc + c0);
          auto acc = [&](int c) -> float { if constexpr (F8) return __uint_as_float(r[c]); else return (float)(int)r[c]; };
          if (p.out_dt == HERO_F8) {
            int8_t* dst = reinterpret_cast<int8_t*>(p.out) + grow * p.out_ld + gcol;
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float4 sc = o4[k];
              const int c = 4 * k;
              w[k] = ptx::f32x4_to_e4m3x4(acc(c) * rowf * sc.x, acc(c + 1) * rowf * sc.y, acc(c + 2) * rowf * sc.z, acc(c + 3) * rowf * sc.w);
            }
            st_g16(dst, w[0], w[1], w[2], w[3]);
          } else if (p.out_dt == HERO_I8) {
            int8_t* dst = reinterpret_cast<int8_t*>(p.out) + grow * p.out_ld + gcol;
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float4 sc = o4[k];
              const int c = 4 * k;
              // Round(acc f) in the FMA's single rounding (magic + x), clipped to [-127, 127] on the shifted value (the
              // order of floats is that of the sums, whatever their size); low byte = two's-complement code
              const float lo = ATT_MAGIC - 127.0f, hi = ATT_MAGIC + 127.0f;
              const float a = fminf(fmaxf(fmaf(acc(c), ROWMAX ? rowf * sc.x : sc.x, ATT_MAGIC), lo), hi);
              const float b = fminf(fmaxf(fmaf(acc(c + 1), ROWMAX ? rowf * sc.y : sc.y, ATT_MAGIC), lo), hi);
              const float cc = fminf(fmaxf(fmaf(acc(c + 2), ROWMAX ? rowf * sc.z : sc.z, ATT_MAGIC), lo), hi);
              const float d = fminf(fmaxf(fmaf(acc(c + 3), ROWMAX ? rowf * sc.w : sc.w, ATT_MAGIC), lo), hi);
              w[k] = low_bytes4_u(a, b, cc, d);
            }
            st_g16(dst, w[0], w[1], w[2], w[3]);
          } else {
            uint16_t* dst = reinterpret_cast<uint16_t*>(p.out) + grow * p.out_ld + gcol;
#pragma unroll
            for (int gq = 0; gq < 2; ++gq) {
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) v[e] = acc(8 * gq + e) * rowf * p.pv_scale;
              st_g16(dst + 8 * gq, fp2(v[0], v[1], p.out_dt), fp2(v[2], v[3], p.out_dt), fp2(v[4], v[5], p.out_dt),
                     fp2(v[6], v[7], p.out_dt));
            }
          }
        }
      }
      ++wcnt;
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == PIPE_QK_WARP) ptx::tmem_dealloc(tmem_base, 512);
}

template <int DH, bool ROWMAX, bool F8, bool PROBE = false>
static hero_status launch_pipe(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream) {
  using Cfg = PipeCfg<DH>;
  const uint64_t rows = (uint64_t)a->B * a->S, cols = (uint64_t)a->nh * DH;
  CUtensorMap tq, tk, tv;
  hero_status st;
  if ((st = make_tmap_2d(h, &tq, a->q, 1, false, false, rows, cols, (uint64_t)a->ld, DH, ATT_BM, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tk, a->k, 1, false, false, rows, cols, (uint64_t)a->ld, DH, PB, DH)) != HERO_OK) return st;
  if ((st = make_tmap_2d(h, &tv, a->v, 1, false, false, rows, cols, (uint64_t)a->ld, DH, PB, DH)) != HERO_OK) return st;
  if (F8) {
    p.idesc_qk = ptx::make_idesc(1, 0, 0, 0, 0, ATT_BM, PB);       // E4M3 x E4M3 -> F32, both K-major
    p.idesc_pv = ptx::make_idesc(1, 0, 0, 0, 1, ATT_BM, DH);       // E4M3 x E4M3 -> F32, V is MN-major
  } else {
    p.idesc_qk = ptx::make_idesc(2, 1, 1, 0, 0, ATT_BM, PB);       // S8 x S8 -> S32
    p.idesc_pv = ptx::make_idesc(2, 0, 1, 0, 1, ATT_BM, DH);       // U8 x S8 -> S32
  }
  auto kern = attn_int8_pipe_kernel<DH, ROWMAX, F8, PROBE>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  const long long tiles = (long long)p.nqt * a->nh * a->B;
  const int grid = (int)(tiles < h->sm_count ? tiles : h->sm_count);
  {
    LaunchScope scope(h, stream, KERNEL_ATTN);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(PIPE_THREADS), Cfg::SMEM_BYTES, stream, tq, tk, tv, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}


hero_status attn_pipe_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream, bool probe) {
  if (probe) {                                               // INT8 operands only (checked by the caller)
    if (a->p_mode == HERO_P_ROWMAX)
      return a->dh == 64 ? launch_pipe<64, true, false, true>(h, a, p, stream) : launch_pipe<128, true, false, true>(h, a, p, stream);
    return a->dh == 64 ? launch_pipe<64, false, false, true>(h, a, p, stream) : launch_pipe<128, false, false, true>(h, a, p, stream);
  }
  if (a->dtype == HERO_F8) {                                 // static P quantizer only (checked by the caller)
    if (a->dh == 64) return launch_pipe<64, false, true>(h, a, p, stream);
    return launch_pipe<128, false, true>(h, a, p, stream);
  }
  if (a->p_mode == HERO_P_ROWMAX) {
    if (a->dh == 64) return launch_pipe<64, true, false>(h, a, p, stream);
    return launch_pipe<128, true, false>(h, a, p, stream);
  }
  if (a->dh == 64) return launch_pipe<64, false, false>(h, a, p, stream);
  return launch_pipe<128, false, false>(h, a, p, stream);
}

}  // namespace hero
