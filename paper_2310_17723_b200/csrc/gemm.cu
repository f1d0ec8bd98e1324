// GeMM^quant (Sec. 2.2.2 Eq. 14, 18, 20-23; Sec. 2.2.3 Eq. 28-30, 32): INT8 x INT8 -> INT32 on the
// tcgen05 tensor cores with the dequantize / bias / GELU / requantize epilogue applied straight
// from tensor memory, plus the FP16/BF16 variant for modules left in FP mode (Table 1).
//
// One persistent CTA per SM, 10 warps:
//   warps 0-7  epilogue: TMEM -> registers -> fused epilogue -> global (warp w owns TMEM lanes 32 (w & 3) ..
//              +31 and the column half w >> 2 of the tile)
//   warp  8    TMA producer: 128-byte-swizzled K-major tiles of A [128 x 128 B] and W [BN x 128 B]
//   warp  9    UMMA issuer (one elected lane) and owner of the TMEM allocation
// The accumulator is double-buffered in TMEM (2 x BN columns) so the epilogue of tile t overlaps the
// main loop of tile t+1.  Every barrier wait is bounded; on expiry the CTA records a code and unwinds.
#include "gemm_common.cuh"

namespace hero {

__device__ __forceinline__ uint32_t pack4_i8(float a, float b, float c, float d) {
  int ia = __float2int_rn(fminf(fmaxf(a, -127.f), 127.f));
  int ib = __float2int_rn(fminf(fmaxf(b, -127.f), 127.f));
  int ic = __float2int_rn(fminf(fmaxf(c, -127.f), 127.f));
  int id = __float2int_rn(fminf(fmaxf(d, -127.f), 127.f));
  return (uint32_t)(ia & 0xff) | ((uint32_t)(ib & 0xff) << 8) | ((uint32_t)(ic & 0xff) << 16) | ((uint32_t)id << 24);
}
// the low bytes of four floats already rounded with ROUND_MAGIC, packed little-endian
__device__ __forceinline__ uint32_t low_bytes4(float a, float b, float c, float d) {
  const uint32_t ab = __byte_perm(__float_as_uint(a), __float_as_uint(b), 0x0040);
  const uint32_t cd = __byte_perm(__float_as_uint(c), __float_as_uint(d), 0x0040);
  return __byte_perm(ab, cd, 0x5410);
}
__device__ __forceinline__ uint32_t pack2_fp(float a, float b, int dt) {
  if (dt == HERO_F16) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void st16(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int& mt, int& nt) {
  // grouped order: consecutive tiles sweep GROUP_M row-tiles of one column-tile strip, so that the
  // tiles in flight at any moment share A and W panels in L2
  constexpr int GROUP_M = 16;
  const int width = GROUP_M * num_n;
  const int group = t / width;
  const int first_m = group * GROUP_M;
  const int gsize = min(num_m - first_m, GROUP_M);
  const int r = t - group * width;
  mt = first_m + (r % gsize);
  nt = r / gsize;
}

// The same order walked tile by tile without integer divisions: the epilogue threads advance by the grid's stride and
// read the coordinates off (group, r); only a last, shorter group of row-tiles needs a division.
struct TileWalk {
  int group, r, width, num_m;
  __device__ __forceinline__ void init(int t, int num_m_, int num_n) {
    num_m = num_m_; width = 16 * num_n; group = t / width; r = t - group * width;
  }
  __device__ __forceinline__ void advance(int stride) {
    r += stride;
    while (r >= width) { r -= width; ++group; }
  }
  __device__ __forceinline__ void coords(int& mt, int& nt) const {
    const int first_m = group * 16, gsize = min(num_m - first_m, 16);
    if (gsize == 16) { mt = first_m + (r & 15); nt = r >> 4; }
    else { mt = first_m + r % gsize; nt = r / gsize; }
  }
};

__device__ __forceinline__ void st32(void* p, const uint32_t (&w)[8]) {   // 256-bit store, 32-byte aligned
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
               "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

// 16 bytes from shared memory through the shared window (a generic load would take the slower generic path)
__device__ __forceinline__ float4 lds_f4(const float* p) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ptx::smem_u32(p)));
  return v;
}

// NC (16 or 32) columns of one output row: v = acc * rs * cs[j] + bias[j];  a = act(v) * post[j];
// INT8: clip(Round(a)) | FP16 / BF16: a | INT32: acc.  Per-column vectors come from shared memory four at a time,
// the arithmetic runs on packed FP32 pairs, the row segment leaves in 32-byte stores when the output allows it.
// How a CTA's 128 x 256 piece of an 8-bit output tile leaves the SM when the epilogue sets the pace (few k-blocks per
// tile).  Straight from registers every lane writes its own row: 32 different 128-byte lines per store instruction,
// which the load/store pipe takes one line at a time.  Instead the epilogue warps put the piece together in shared
// memory (two halves of 128 rows x 128 bytes in the tensor map's 128-byte swizzle, so that the lanes' 16-byte writes
// spread over all banks) and meet a store warp on a named barrier; its elected lane hands each half to the TMA unit as a
// bulk tensor store, which also clips rows and columns beyond the matrix, waits until the unit has read the tile and
// then arrives on a second named barrier, which the epilogue warps pass before their first write of the next tile
// (long after, as a rule).  The staging area is the pipeline's last stage, which a launch of this kind leaves unused
// (five stages feed a short main loop as well as six).
struct OutStage {
  uint8_t* buf;               // the CTA's staging tile (NULL: direct stores)
  const CUtensorMap* tm;      // box = 128 rows x 128 bytes
  uint32_t lane_off;          // this lane's row: byte offset of the row in a half, and its swizzle term
  uint32_t lane_sw;
  int n0;                     // first column of the tile being processed
  bool fresh;                 // nothing of the current tile has been staged yet
  int nthreads;               // threads on the two named barriers: epilogue warps + store warp
  int bar_staged, bar_drained;   // named barriers of this warp's group: tile staged (epilogue -> store warp), tile read (back)
  bool clip_low;              // GELU: some output factor of this warp's columns is negative or above 700, so that
                              // GELU(v) * factor >= -0.17 * factor may fall below -127 (otherwise only the upper clip can bite)
};
constexpr int BAR_STAGED = 1, BAR_DRAINED = 3;   // first named barrier of each kind (+ the epilogue group's index)
constexpr int OUT_HALF_BYTES = GEMM_BM * 128;
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_2d(const CUtensorMap* tm, const void* smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(ptx::smem_u32(smem_src)) : "memory");
}
__device__ __forceinline__ void bulk_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void sts16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <bool INT8, int ACT, int OUTK, int NC>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, const uint32_t (&r)[NC], const float* e_cs,
                                               const float* e_bias, const float* e_post, int m, bool row_ok, float rs,
                                               int col0, bool wide, OutStage& stage) {
  if constexpr (OUTK == OUT_I32) {
    if (!row_ok) return;
    int* dst = reinterpret_cast<int*>(p.out) + (long long)m * p.out_ld + col0;
    if (wide && col0 + NC <= p.N) {
#pragma unroll
      for (int g = 0; g < NC / 8; ++g) {
        const uint32_t w[8] = {r[8 * g], r[8 * g + 1], r[8 * g + 2], r[8 * g + 3], r[8 * g + 4], r[8 * g + 5], r[8 * g + 6], r[8 * g + 7]};
        st32(dst + 8 * g, w);
      }
    } else {
#pragma unroll
      for (int g = 0; g < NC / 4; ++g)
        if (col0 + 4 * g + 4 <= p.N) st16(dst + 4 * g, r[4 * g], r[4 * g + 1], r[4 * g + 2], r[4 * g + 3]);
    }
  } else {
    float v[NC];
    float hi = -INFINITY, lo = INFINITY;
    const float2 rs2 = make_float2(rs, rs), mg2 = make_float2(ROUND_MAGIC, ROUND_MAGIC);
#pragma unroll
    for (int j = 0; j < NC; j += 4) {
      const float4 cs4 = lds_f4(e_cs + j), b4 = lds_f4(e_bias + j);
      float2 a0, a1;
      if constexpr (INT8) {
        a0 = make_float2((float)(int)r[j], (float)(int)r[j + 1]);
        a1 = make_float2((float)(int)r[j + 2], (float)(int)r[j + 3]);
      } else {
        a0 = make_float2(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
        a1 = make_float2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      }
      float2 x0 = __ffma2_rn(__fmul2_rn(a0, rs2), make_float2(cs4.x, cs4.y), make_float2(b4.x, b4.y));
      float2 x1 = __ffma2_rn(__fmul2_rn(a1, rs2), make_float2(cs4.z, cs4.w), make_float2(b4.z, b4.w));
      float2 y0, y1;
      if constexpr (ACT == HERO_ACT_NONE) {
        // without an activation the output factor is already folded into cs and bias (see epilogue_loop)
        if constexpr (OUTK == OUT_I8) { y0 = __fadd2_rn(x0, mg2); y1 = __fadd2_rn(x1, mg2); }
        else { y0 = x0; y1 = x1; }                          // FP and e4m3 outputs: the conversion rounds
      } else {
        const float4 p4 = lds_f4(e_post + j);
        if constexpr (ACT == HERO_ACT_GELU_ERF) { x0 = gelu_erf_f2(x0); x1 = gelu_erf_f2(x1); }
        if constexpr (ACT == HERO_ACT_GELU_TANH) {
          x0.x = gelu_tanh_f(x0.x); x0.y = gelu_tanh_f(x0.y); x1.x = gelu_tanh_f(x1.x); x1.y = gelu_tanh_f(x1.y);
        }
        if constexpr (OUTK == OUT_I8) {
          y0 = __ffma2_rn(x0, make_float2(p4.x, p4.y), mg2);
          y1 = __ffma2_rn(x1, make_float2(p4.z, p4.w), mg2);
        } else {
          y0 = __fmul2_rn(x0, make_float2(p4.x, p4.y));
          y1 = __fmul2_rn(x1, make_float2(p4.z, p4.w));
        }
      }
      v[j] = y0.x; v[j + 1] = y0.y; v[j + 2] = y1.x; v[j + 3] = y1.y;
      if constexpr (OUTK == OUT_I8) {
        // Round (half to even) happened in the float adder: 1.5 * 2^23 + k keeps k in its low byte.  The clip to
        // [-127, 127] is applied only if some value of the chunk needs it.
        hi = ptx::max3(ptx::max3(hi, y0.x, y0.y), y1.x, y1.y);
        if constexpr (ACT == HERO_ACT_NONE) lo = ptx::min3(ptx::min3(lo, y0.x, y0.y), y1.x, y1.y);
      }
    }
    if constexpr (OUTK == OUT_I8) {
      // (after a GELU the lower bound is known from the output factors alone: see OutStage::clip_low)
      if (hi > ROUND_MAGIC + 127.0f || (ACT == HERO_ACT_NONE ? lo < ROUND_MAGIC - 127.0f : stage.clip_low)) {
#pragma unroll
        for (int j = 0; j < NC; ++j) v[j] = fminf(fmaxf(v[j], ROUND_MAGIC - 127.0f), ROUND_MAGIC + 127.0f);
      }
    }
    if constexpr (OUTK == OUT_I8 || OUTK == OUT_F8) {
      uint32_t w[NC / 4];
#pragma unroll
      for (int g = 0; g < NC / 4; ++g) {
        if constexpr (OUTK == OUT_F8) w[g] = ptx::f32x4_to_e4m3x4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);   // saturating RNE
        else w[g] = low_bytes4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
      }
      if (stage.buf) {
        // this lane's NC bytes of its row of the staging tile (rows past the end are clipped by the store)
        if (stage.fresh) {                                   // the unit has read the previous tile out of the staging area
          asm volatile("bar.sync %0, %1;" ::"r"(stage.bar_drained), "r"(stage.nthreads) : "memory");
          stage.fresh = false;
        }
        const int jc = col0 - stage.n0;                      // column inside the tile
        const uint32_t half = ptx::smem_u32(stage.buf) + (jc >> 7) * OUT_HALF_BYTES + stage.lane_off;
        const uint32_t c16 = (jc & 127) >> 4;
        sts16(half + (((c16) ^ stage.lane_sw) << 4), w[0], w[1], w[2], w[3]);
        if constexpr (NC == 32) sts16(half + (((c16 + 1) ^ stage.lane_sw) << 4), w[4], w[5], w[6], w[7]);
        return;
      }
      if (!row_ok) return;
      int8_t* dst = reinterpret_cast<int8_t*>(p.out) + (long long)m * p.out_ld + col0;
      if constexpr (NC == 32) {
        if (wide && col0 + 32 <= p.N) {
          st32(dst, w);
        } else {
          if (col0 + 16 <= p.N) st16(dst, w[0], w[1], w[2], w[3]);
          if (col0 + 32 <= p.N) st16(dst + 16, w[4], w[5], w[6], w[7]);
        }
      } else {
        if (col0 + 16 <= p.N) st16(dst, w[0], w[1], w[2], w[3]);
      }
    } else {
      uint32_t w[NC / 2];
#pragma unroll
      for (int g = 0; g < NC / 2; ++g) w[g] = pack2_fp(v[2 * g], v[2 * g + 1], p.out_dt);
      if (p.obs_col) {
        // calibration observer: the absolute maximum of every column of this piece over the warp's 32 rows, taken from
        // the values as stored (non-negative floats order like their bit patterns: an integer warp reduction and an
        // integer atomic maximum do), lane c reporting column c
        const int lane = threadIdx.x & 31;
        uint32_t mine = 0;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const uint32_t h16 = (w[c >> 1] >> (16 * (c & 1))) & 0x7fffu;          // |x| in the stored 16-bit type
          const float ax = p.out_dt == HERO_F16 ? __half2float(__ushort_as_half((unsigned short)h16)) : __uint_as_float(h16 << 16);
          const uint32_t mx = __reduce_max_sync(0xffffffffu, row_ok ? __float_as_uint(ax) : 0u);
          if (lane == c) mine = mx;
        }
        if (lane < NC && col0 + lane < p.N && mine != 0u) atomicMax(reinterpret_cast<unsigned int*>(p.obs_col) + col0 + lane, mine);
      }
      if (!row_ok) return;
      uint16_t* dst = reinterpret_cast<uint16_t*>(p.out) + (long long)m * p.out_ld + col0;
      if (wide && col0 + NC <= p.N) {
#pragma unroll
        for (int g = 0; g < NC / 16; ++g) {
          const uint32_t w0[8] = {w[8 * g], w[8 * g + 1], w[8 * g + 2], w[8 * g + 3], w[8 * g + 4], w[8 * g + 5], w[8 * g + 6], w[8 * g + 7]};
          st32(dst + 16 * g, w0);
        }
      } else {
#pragma unroll
        for (int g = 0; g < NC / 8; ++g)
          if (col0 + 8 * g + 8 <= p.N) st16(dst + 8 * g, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
      }
    }
  }
}

// One thread's share of a tile's epilogue: BN / (EW / 4) columns of one output row (EW epilogue warps, EW / 4 per
// tensor-memory lane quarter).  With 8 warps the columns come 32 at a time, the next 32 already loading while the
// current ones are processed; with 16 warps (96 registers per thread) 16 at a time.
template <int BN, bool INT8, int ACT, int OUTK, int CH, int CW>
__device__ __forceinline__ void epilogue_columns(const GemmParams& p, const float* e_cs, const float* e_bias,
                                                 const float* e_post, uint32_t taddr, int m, bool row_ok, float rs,
                                                 int n0, int cpart, OutStage& stage) {
  // 32-byte stores need a 32-byte aligned row segment: base pointer and row pitch multiples of 32 bytes
  const int es = (OUTK == OUT_I8 || OUTK == OUT_F8) ? 1 : (OUTK == OUT_FP ? 2 : 4);
  const bool wide = ((reinterpret_cast<uintptr_t>(p.out) & 31) == 0) && ((p.out_ld * es) % 32 == 0);
  if constexpr (CW == 32) {
    constexpr int NCH = CH / 32;
    uint32_t ra[32], rb[32];
    ptx::tmem_ld32(taddr, ra);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      ptx::tmem_ld_wait();
      if (c + 1 < NCH) ptx::tmem_ld32(taddr + (c + 1) * 32, (c & 1) ? ra : rb);
      const int jw = c * 32;                // column of the chunk's first element among this warp's columns
      const int jc = cpart * CH + jw;       // ... and inside the tile
      if (c & 1) epilogue_chunk<INT8, ACT, OUTK, 32>(p, rb, e_cs + jw, e_bias + jw, e_post + jw, m, row_ok, rs, n0 + jc, wide, stage);
      else epilogue_chunk<INT8, ACT, OUTK, 32>(p, ra, e_cs + jw, e_bias + jw, e_post + jw, m, row_ok, rs, n0 + jc, wide, stage);
    }
  } else {
    constexpr int NCH = CH / 16;
    uint32_t ra[16], rb[16];
    ptx::tmem_ld16(taddr, ra);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      ptx::tmem_ld_wait();
      if (c + 1 < NCH) ptx::tmem_ld16(taddr + (c + 1) * 16, (c & 1) ? ra : rb);
      const int jw = c * 16;
      const int jc = cpart * CH + jw;
      if (c & 1) epilogue_chunk<INT8, ACT, OUTK, 16>(p, rb, e_cs + jw, e_bias + jw, e_post + jw, m, row_ok, rs, n0 + jc, wide, stage);
      else epilogue_chunk<INT8, ACT, OUTK, 16>(p, ra, e_cs + jw, e_bias + jw, e_post + jw, m, row_ok, rs, n0 + jc, wide, stage);
    }
  }
}

// The epilogue warps' walk over this CTA's tiles.  The per-column vectors (and the row scale) of the NEXT tile are
// fetched from global memory into registers while the current tile is being processed, so a tile never starts by
// waiting on them.  ROWS = output rows per tile (128, or 256 for a CTA pair of which this CTA owns rows row_off..+127).
// GROUPS = 2 (16 epilogue warps with a staged output): the warps form two groups of eight that take alternate tiles, each
// group always the same accumulator buffer and its own staging tile.  The two groups are then half a tile apart in time:
// while one group's warps wait (for tensor memory, for their barrier) the other's keep the issue slots busy, which 16
// warps moving through the same chunk in step do not.
template <int BN, bool INT8, int ACT, int OUTK, int ROWS, bool PAIR, int EW, int GROUPS = 1>
__device__ __forceinline__ void epilogue_loop(const GemmParams& p, float* epi, uint64_t* acc_full, uint64_t* acc_empty,
                                              uint32_t tmem_base, int first_tile, int tile_stride, int row_off,
                                              OutStage stage, int warp) {   // warp: index among the epilogue warps
  const int lane = threadIdx.x & 31;
  constexpr int EWG = EW / GROUPS;           // warps per group
  constexpr int CH = BN / (EWG / 4);         // columns per thread and tile
  constexpr int CW = EW == 8 ? 32 : 16;      // columns per chunk (registers: 8 warps afford 32, 16 warps 16)
  const int wg = warp / EWG, wl = warp % EWG;
  const int quarter = warp & 3, cpart = wl >> 2;
  const int num_tiles = p.num_m_tiles * p.num_n_tiles;
  bool ok = true;
  first_tile += wg * tile_stride;            // this group's tiles: every GROUPS-th of the CTA's
  tile_stride *= GROUPS;

  // Every warp stages the per-column vectors of its own CH columns in a shared-memory area of its own (3 x CH floats:
  // written at the start of a tile, after the warp's last read of the previous tile's), so the epilogue warps never
  // wait for one another.
  constexpr int NV = CH / 32;                // values per lane and vector
  float* epi_w = epi + warp * (3 * CH);
  float ncs[NV], nbias[NV], npost[NV], nrs = 1.0f;
  TileWalk walk;                             // stands at the tile whose vectors are fetched next
  walk.init(first_tile, p.num_m_tiles, p.num_n_tiles);
  int nmt = 0, nnt = 0;                      // its coordinates, consumed one tile later like the vectors
  auto fetch = [&]() {                       // issue the loads for the walker's tile, then step on
    int mt, nt; walk.coords(mt, nt);
    nmt = mt; nnt = nt;
    walk.advance(tile_stride);
    if constexpr (OUTK != OUT_I32) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int n = nt * BN + cpart * CH + i * 32 + lane;
        const bool in = n < p.N;
        ncs[i] = (in && p.cs) ? __ldg(p.cs + n) : 1.0f;
        nbias[i] = (in && p.bias) ? __ldg(p.bias + n) : 0.0f;
        npost[i] = (in && p.post) ? __ldg(p.post + n) : 1.0f;
      }
      const int m = mt * ROWS + row_off + quarter * 32 + lane;
      nrs = (p.rs && m < p.M) ? __ldg(p.rs + m) : 1.0f;
    }
  };
  auto publish = [&](int it) {               // registers -> this tile's shared-memory vectors
    if constexpr (OUTK != OUT_I32) {
      float* e = epi_w;
      __syncwarp();                          // every lane is through with the previous tile's vectors
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        if constexpr (ACT == HERO_ACT_NONE) {    // (acc rs cs + b) post = acc rs (cs post) + b post
          e[i * 32 + lane] = ncs[i] * npost[i]; e[CH + i * 32 + lane] = nbias[i] * npost[i];
        } else {
          e[i * 32 + lane] = ncs[i]; e[CH + i * 32 + lane] = nbias[i]; e[2 * CH + i * 32 + lane] = npost[i];
        }
      }
      if constexpr (ACT != HERO_ACT_NONE) {
        bool odd = false;
#pragma unroll
        for (int i = 0; i < NV; ++i) odd = odd || !(npost[i] >= 0.0f && npost[i] <= 700.0f);
        stage.clip_low = __any_sync(0xffffffffu, odd);
      }
      __syncwarp();
    }
  };

  if (first_tile < num_tiles) fetch();
  int it = 0;
  for (int t = first_tile; t < num_tiles; t += tile_stride, ++it) {
    const int mt = nmt, nt = nnt;
    const int as = GROUPS == 2 ? wg : (it & 1);
    const uint32_t aphase = GROUPS == 2 ? (it & 1) : ((it >> 1) & 1);
    const int n0 = nt * BN;
    const float rs = nrs;
    publish(it);
    if (t + tile_stride < num_tiles) fetch();
    const float* e_cs = epi_w;
    const int m = mt * ROWS + row_off + quarter * 32 + lane;
    const bool row_ok = m < p.M;

    // a wait that gave up has recorded its code; the warp runs on without waiting again so that the kernel ends promptly
    if (ok && !ptx::mbar_wait(&acc_full[as], aphase, p.err, 0x400 | as)) ok = false;
    ptx::tc_fence_after();
    stage.n0 = n0;
    stage.fresh = it > 0;                                  // (the first tile finds the staging area unused)
    {
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + as * BN + cpart * CH;
      epilogue_columns<BN, INT8, ACT, OUTK, CH, CW>(p, e_cs, e_cs + CH, e_cs + 2 * CH, taddr, m, row_ok, rs, n0, cpart, stage);
    }
    // hand the accumulator buffer back to the UMMA issuer
    ptx::tc_fence_before();
    __syncwarp();
    if (lane == 0) {
      if constexpr (PAIR) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(ptx::smem_u32(&acc_empty[as]), 0));
      else ptx::mbar_arrive(&acc_empty[as]);
    }
    if (stage.buf) {
      // this warp's part of the staged tile is complete (writes made visible to the TMA unit)
      ptx::fence_proxy_async_smem();
      asm volatile("bar.sync %0, %1;" ::"r"(stage.bar_staged), "r"(stage.nthreads) : "memory");
    }
  }
}

template <int BN, bool INT8, int ACT, int OUTK>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const GemmParams p) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* tiles = smem;
  float* epi = reinterpret_cast<float*>(smem + STAGES * Cfg::STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi + Cfg::EPI_FLOATS);
  uint64_t* full = bars;                    // [STAGES]  TMA -> MMA
  uint64_t* empty = bars + STAGES;          // [STAGES]  MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;   // [2]       MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;       // [2]       epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.num_m_tiles * p.num_n_tiles;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&full[i], 1); ptx::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 8); }
    ptx::fence_mbar_init();
  }
  if (warp == MMA_WARP) {
    ptx::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  if (warp == TMA_WARP && lane == 0) { ptx::prefetch_tmap(&tmA); ptx::prefetch_tmap(&tmW); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch_dependents();

  if (warp == TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer
    // (this loop and the UMMA issuer's are walked by the whole warp, one elected lane issuing: uniform control flow keeps
    // the addresses in the uniform datapath, and these serial chains have to keep up with the tensor core)
    {
      const bool issue = ptx::elect_one();
      const int kelems = GEMM_BK_BYTES / p.elem_bytes;
      int stage = 0; uint32_t phase = 0; bool ok = true;
      // The weights are constants of the model: the W tiles of the first tile's first stages are requested before the
      // dependency wait, the activation tiles after it (both complete the same barrier).
      int pre = 0;
      if ((int)blockIdx.x < num_tiles) {
        int mt, nt; tile_coords(blockIdx.x, p.num_m_tiles, p.num_n_tiles, mt, nt);
        pre = min(p.num_kb, STAGES);
        if (issue) {
          for (int kb = 0; kb < pre; ++kb) {
            ptx::mbar_expect_tx(&full[kb], Cfg::STAGE_BYTES);
            ptx::tma_load_2d(tiles + kb * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tmW, kb * kelems, nt * BN, &full[kb]);
          }
        }
      }
      ptx::pdl_wait();                                   // the previous kernel's outputs are complete and visible from here on
      bool first = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        int mt, nt; tile_coords(t, p.num_m_tiles, p.num_n_tiles, mt, nt);
        const int ya = mt * GEMM_BM, yw = nt * BN;
        int x = 0;
        for (int kb = 0; kb < p.num_kb; ++kb, x += kelems) {
          const bool early = first && kb < pre;          // barrier armed and W requested above
          if (!early && !ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x100 | stage)) { ok = false; break; }
          if (issue) {
            uint8_t* a_dst = tiles + stage * Cfg::STAGE_BYTES;
            if (!early) ptx::mbar_expect_tx(&full[stage], Cfg::STAGE_BYTES);
            ptx::tma_load_2d(a_dst, &tmA, x, ya, &full[stage]);
            if (!early) ptx::tma_load_2d(a_dst + Cfg::A_BYTES, &tmW, x, yw, &full[stage]);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        first = false;
      }
      // drain: every copy this thread started has landed before the CTA may exit
      for (int i = 0; i < STAGES; ++i) {
        if (!ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x180 | stage)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == MMA_WARP) {
    // ------------------------------------------------------------------ UMMA issuer
    ptx::pdl_wait();
    {
      const bool issue = ptx::elect_one();
      constexpr uint64_t desc_base = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);
      // descriptors differ only in the start-address field (address >> 4): one base per operand, small additions later
      const uint64_t ad0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles));
      const uint64_t bd0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles) + Cfg::A_BYTES);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (it >> 1) & 1;
        if (!ptx::mbar_wait(&acc_empty[as], aphase ^ 1, p.err, 0x200 | as)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!ptx::mbar_wait(&full[stage], phase, p.err, 0x300 | stage)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint32_t so = (uint32_t)(stage * Cfg::STAGE_BYTES) >> 4;
#pragma unroll
            for (int k = 0; k < GEMM_BK_BYTES / 32; ++k) {
              const uint64_t ad = ad0 + (so + 2 * k), bd = bd0 + (so + 2 * k);
              if constexpr (INT8) ptx::umma_i8(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
              else if (p.f8) ptx::umma_f8(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
              else ptx::umma_f16(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
            }
            ptx::umma_commit(&empty[stage]);    // frees the smem stage once these MMAs have read it
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok && issue) ptx::umma_commit(&acc_full[as]);  // accumulator of this tile complete
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-7)
    // warp w reads TMEM lanes 32 * (w & 3) .. +31 (one output row per thread) and the column half (w >> 2)
    ptx::pdl_wait();                                     // before this warp's first global access
    epilogue_loop<BN, INT8, ACT, OUTK, GEMM_BM, false, 8>(p, epi, acc_full, acc_empty, tmem_base, blockIdx.x, gridDim.x, 0,
                                                           OutStage{nullptr, nullptr, 0, 0, 0, false, 0, 0, 0, true}, warp);
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == MMA_WARP) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
}

template <int BN, bool INT8, int ACT, int OUTK>
static hero_status launch_gemm(hero_handle* h, const CUtensorMap& tmA, const CUtensorMap& tmW, const GemmParams& p,
                               cudaStream_t stream) {
  using Cfg = GemmCfg<BN>;
  auto kern = gemm_kernel<BN, INT8, ACT, OUTK>;
  HERO_SMEM_OPT_IN(h, kern, Cfg::SMEM_BYTES);
  const int tiles = p.num_m_tiles * p.num_n_tiles;
  const int grid = tiles < h->sm_count ? tiles : h->sm_count;
  {
    LaunchScope scope(h, stream, KERNEL_GEMM);
    HERO_CUDA(launch_dependent(kern, dim3(grid), dim3(GEMM_THREADS), Cfg::SMEM_BYTES, stream, tmA, tmW, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

template <int BN, bool INT8>
static hero_status dispatch_epilogue(hero_handle* h, const CUtensorMap& tmA, const CUtensorMap& tmW, const GemmParams& p,
                                     int act, cudaStream_t s) {
  if (p.out_dt == HERO_I32) {
    if constexpr (INT8) return launch_gemm<BN, true, HERO_ACT_NONE, OUT_I32>(h, tmA, tmW, p, s);
    else { set_error("raw INT32 output needs INT8 operands"); return HERO_ERR_UNSUPPORTED; }
  }
  if (p.out_dt == HERO_F8) {
    if constexpr (!INT8) {
      switch (act) {
        case HERO_ACT_NONE: return launch_gemm<BN, false, HERO_ACT_NONE, OUT_F8>(h, tmA, tmW, p, s);
        case HERO_ACT_GELU_ERF: return launch_gemm<BN, false, HERO_ACT_GELU_ERF, OUT_F8>(h, tmA, tmW, p, s);
        case HERO_ACT_GELU_TANH: return launch_gemm<BN, false, HERO_ACT_GELU_TANH, OUT_F8>(h, tmA, tmW, p, s);
      }
    }
    set_error("an e4m3 output needs e4m3 or FP operands");
    return HERO_ERR_UNSUPPORTED;
  }
  const bool i8 = p.out_dt == HERO_I8;
  switch (act) {
    case HERO_ACT_NONE:
      return i8 ? launch_gemm<BN, INT8, HERO_ACT_NONE, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm<BN, INT8, HERO_ACT_NONE, OUT_FP>(h, tmA, tmW, p, s);
    case HERO_ACT_GELU_ERF:
      return i8 ? launch_gemm<BN, INT8, HERO_ACT_GELU_ERF, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm<BN, INT8, HERO_ACT_GELU_ERF, OUT_FP>(h, tmA, tmW, p, s);
    case HERO_ACT_GELU_TANH:
      return i8 ? launch_gemm<BN, INT8, HERO_ACT_GELU_TANH, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm<BN, INT8, HERO_ACT_GELU_TANH, OUT_FP>(h, tmA, tmW, p, s);
  }
  set_error("unknown activation %d", act);
  return HERO_ERR_INVALID_ARG;
}

// ------------------------------------------------------------------------------------------------------
// CTA-pair variant (tcgen05 cta_group::2): two CTAs of a cluster share one 256 x 256 tile.  Each CTA loads its
// own 128 rows of A and its own 128 of the 256 W rows (32 KB per k-block instead of 48 KB for the same number
// of MACs per SM, which is what the L2 -> SM path limits), the leader CTA's elected lane issues M = 256 UMMAs
// that read both CTAs' shared memory, and each CTA's tensor memory receives its 128 accumulator rows.
//   full[s]      (leader's copy) : each CTA's producer loads its own two half-tiles into its own shared memory; all
//                                  four copies complete on this barrier, which the leader arms with the total byte count
//   empty[s]     (every CTA)     : the leader's commit is multicast to both CTAs (each producer waits on its own copy)
//   acc_full[a]  (every CTA)     : the leader's commit is multicast to both CTAs
//   acc_empty[a] (leader's copy) : all epilogue warps of the pair arrive on it
// The two single-lane loops (producer, UMMA issuer) are serial chains that must turn a k-block around every ~500 cycles
// beside the epilogue warps: they are kept short (loop-invariant addresses and descriptors computed once, uniform
// control flow) and the copies are split between the two CTAs' producers.
// No multicast TMA load is used anywhere.
// ------------------------------------------------------------------------------------------------------
// The store warp of a launch with staged output: for every tile of this CTA, in the epilogue warps' order (tile i belongs to
// epilogue group i % groups, which has its own staging tile and barrier pair), wait until the tile is staged, send its two
// halves, wait until the unit has read them, tell that group.
template <int ROWS>
__device__ __forceinline__ void store_warp_loop(const GemmParams& p, const CUtensorMap* tm, uint8_t* buf, int first_tile,
                                                int tile_stride, int row_off, int nthreads, int groups) {
  const int num_tiles = p.num_m_tiles * p.num_n_tiles;
  const bool issue = ptx::elect_one();
  TileWalk walk;
  walk.init(first_tile, p.num_m_tiles, p.num_n_tiles);
  int it = 0;
  for (int t = first_tile; t < num_tiles; t += tile_stride, ++it) {
    int mt, nt; walk.coords(mt, nt);
    walk.advance(tile_stride);
    const int g = groups == 2 ? (it & 1) : 0;
    uint8_t* tile = buf + g * 2 * OUT_HALF_BYTES;
    asm volatile("bar.sync %0, %1;" ::"r"(BAR_STAGED + g), "r"(nthreads) : "memory");
    if (issue) {
      const int m0 = mt * ROWS + row_off, n0 = nt * 256;
      if (m0 < p.M) {
        bulk_store_2d(tm, tile, n0, m0);
        if (n0 + 128 < p.N) bulk_store_2d(tm, tile + OUT_HALF_BYTES, n0 + 128, m0);
      }
      bulk_store_commit();
      bulk_store_wait_read();
    }
    __syncwarp();
    if (t + groups * tile_stride < num_tiles) asm volatile("bar.arrive %0, %1;" ::"r"(BAR_DRAINED + g), "r"(nthreads) : "memory");
  }
  if (issue) bulk_store_wait_all();                          // the unit is through with this CTA's shared memory
}

struct PairCfg {
  static constexpr int BN = 256;
  static constexpr int A_BYTES = GEMM_BM * GEMM_BK_BYTES;        // this CTA's 128 rows of A
  static constexpr int B_BYTES = (BN / 2) * GEMM_BK_BYTES;       // this CTA's 128 rows of W
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = 6;
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int EPI_FLOATS = 2 * 4 * 3 * BN;              // per-warp cs / bias / post (two groups of 8 warps: 128 columns each)
  static_assert(STAGE_BYTES == 2 * OUT_HALF_BYTES, "the last stages double as output staging tiles");
  static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + EPI_FLOATS * 4 + 256;
};

template <bool INT8, int ACT, int OUTK, int EW>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__((EW + 3) * 32, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmO, const GemmParams p) {
  using Cfg = PairCfg;
  constexpr int BN = Cfg::BN;
  // with staged output the last pipeline stage is the staging tile; 16 epilogue warps work as two groups with a staging
  // tile each (the last two stages)
  const int groups = (p.tma_out && EW == 16) ? 2 : 1;
  const int STAGES = p.tma_out ? Cfg::STAGES - groups : Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* tiles = smem;
  uint8_t* out_stage = smem + (Cfg::STAGES - groups) * Cfg::STAGE_BYTES;
  float* epi = reinterpret_cast<float*>(smem + Cfg::STAGES * Cfg::STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi + Cfg::EPI_FLOATS);
  uint64_t* full = bars;
  uint64_t* empty = bars + Cfg::STAGES;
  uint64_t* acc_full = bars + 2 * Cfg::STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr int W_TMA = EW, W_MMA = EW + 1, W_ST = EW + 2;   // warps 0 .. EW-1: epilogue; W_ST: store warp (staged output)
  const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
  const int num_tiles = p.num_m_tiles * p.num_n_tiles;   // 256 x 256 tiles
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < Cfg::STAGES; ++i) { ptx::mbar_init(&full[i], 1); ptx::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_empty[i], 2 * EW / groups); }
    ptx::fence_mbar_init();
  }
  if (warp == W_MMA) {
    ptx::tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  if (warp == W_TMA && lane == 0) { ptx::prefetch_tmap(&tmA); ptx::prefetch_tmap(&tmW); if (p.tma_out) ptx::prefetch_tmap(&tmO); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();                                   // both CTAs' barriers exist before any remote arrive
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  ptx::pdl_launch_dependents();

  if (warp == W_TMA) {
    // ------------------------------------------------------------------ TMA producer (one in each CTA of the pair)
    // Each CTA's producer loads its own halves of A and W into its own shared memory; all four copies of a k-block
    // complete on the LEADER's `full` barrier (the leader arms it with the byte count of both CTAs; bytes that land
    // before the arming only run the count negative for a moment).  A CTA's stage is free when the leader's commit,
    // multicast to both CTAs, has arrived on its own `empty` barrier.  One thread can start a bulk tensor copy only
    // every ~90 cycles: four copies per k-block from one thread took most of the ~500 cycles a k-block lasts on the
    // tensor core, two from each of two threads run side by side.
    // The whole warp walks the loop (uniform control flow: the addresses stay in the uniform datapath) and one elected
    // lane issues; everything that does not change from one k-block to the next is computed once.
    {
      const bool issue = ptx::elect_one();
      const int kelems = GEMM_BK_BYTES / p.elem_bytes;
      // cluster addresses are linear in the offset: one mapping for this CTA's tiles, one for the leader's barriers
      const uint32_t dst = ptx::mapa(ptx::smem_u32(tiles), rank);
      const uint32_t bar0 = ptx::mapa(ptx::smem_u32(&full[0]), 0);
      const int ra = (int)rank * GEMM_BM, rw = (int)rank * (BN / 2);   // this CTA's rows of the A and W tiles
      int stage = 0; uint32_t phase = 0; bool ok = true;
      // The weights are constants of the model: the W halves of the first tile's first stages are requested before the
      // dependency wait, the activation halves after it (all complete the same barrier).
      int pre = 0;
      if (pair_id < num_tiles) {
        int mt, nt; tile_coords(pair_id, p.num_m_tiles, p.num_n_tiles, mt, nt);
        pre = min(p.num_kb, STAGES);
        if (issue) {
          for (int kb = 0; kb < pre; ++kb) {
            if (rank == 0) ptx::mbar_expect_tx(&full[kb], 2 * Cfg::STAGE_BYTES);
            ptx::tma_load_2d_pair(dst + kb * Cfg::STAGE_BYTES + Cfg::A_BYTES, &tmW, kb * kelems, nt * BN + rw, bar0 + 8 * kb);
          }
        }
      }
      ptx::pdl_wait();                                   // the previous kernel's outputs are complete and visible from here on
      bool first = true;
      for (int t = pair_id; t < num_tiles && ok; t += num_pairs) {
        int mt, nt; tile_coords(t, p.num_m_tiles, p.num_n_tiles, mt, nt);
        const int ya = mt * 256 + ra, yw = nt * BN + rw;
        int x = 0;
        for (int kb = 0; kb < p.num_kb; ++kb, x += kelems) {
          const bool early = first && kb < pre;          // barrier armed and W requested above
          if (!early && !ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x700 | stage)) { ok = false; break; }
          if (issue) {
            const uint32_t off = stage * Cfg::STAGE_BYTES;
            const uint32_t bar = bar0 + 8 * stage;
            if (!early && rank == 0) ptx::mbar_expect_tx(&full[stage], 2 * Cfg::STAGE_BYTES);
            ptx::tma_load_2d_pair(dst + off, &tmA, x, ya, bar);
            if (!early) ptx::tma_load_2d_pair(dst + off + Cfg::A_BYTES, &tmW, x, yw, bar);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        first = false;
      }
      for (int i = 0; i < STAGES; ++i) {                 // drain: every copy started here has been consumed
        if (!ptx::mbar_wait(&empty[stage], phase ^ 1, p.err, 0x780 | stage)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == W_MMA) {
    // ------------------------------------------------------------------ UMMA issuer (leader CTA only)
    ptx::pdl_wait();
    if (rank == 0) {
      const bool issue = ptx::elect_one();
      constexpr uint64_t desc_base = ptx::smem_desc_base(16, 1024, ptx::SWZ_128B);
      // descriptors differ from stage to stage and k-slice to k-slice only in the start-address field (address >> 4,
      // far from overflowing its 14 bits): one base per operand, small additions afterwards
      const uint64_t ad0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles));
      const uint64_t bd0 = ptx::smem_desc(desc_base, ptx::smem_u32(tiles) + Cfg::A_BYTES);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      int it = 0;
      for (int t = pair_id; t < num_tiles && ok; t += num_pairs, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (it >> 1) & 1;
        if (!ptx::mbar_wait(&acc_empty[as], aphase ^ 1, p.err, 0x800 | as)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!ptx::mbar_wait(&full[stage], phase, p.err, 0x900 | stage)) { ok = false; break; }
          ptx::tc_fence_after();
          if (issue) {
            const uint32_t so = (uint32_t)(stage * Cfg::STAGE_BYTES) >> 4;
#pragma unroll
            for (int k = 0; k < GEMM_BK_BYTES / 32; ++k) {
              const uint64_t ad = ad0 + (so + 2 * k), bd = bd0 + (so + 2 * k);
              if constexpr (INT8) ptx::umma_i8_pair(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
              else if (p.f8) ptx::umma_f8_pair(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
              else ptx::umma_f16_pair(d_tmem, ad, bd, p.idesc, (kb | k) != 0);
            }
            ptx::umma_commit_pair(&empty[stage], 3);     // frees this stage in both CTAs
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok && issue) ptx::umma_commit_pair(&acc_full[as], 3);  // both CTAs' accumulator halves are complete
      }
    }
    __syncwarp();
  } else if (warp == W_ST) {
    // ------------------------------------------------------------------ store warp
    if (p.tma_out) store_warp_loop<256>(p, &tmO, out_stage, pair_id, num_pairs, (int)rank * GEMM_BM, (EW / groups + 1) * 32, groups);
  } else {
    ptx::pdl_wait();                                     // before this warp's first global access
    // ------------------------------------------------------------------ epilogue (warps 0 .. EW-1 of each CTA)
    const int row = (warp & 3) * 32 + lane;                // this lane's row of the CTA's 128
    const int wg = groups == 2 ? warp / (EW / 2) : 0;      // this warp's epilogue group
    OutStage stage{p.tma_out ? out_stage + wg * 2 * OUT_HALF_BYTES : nullptr, &tmO, (uint32_t)row * 128u, (uint32_t)row & 7u, 0, false,
                   (EW / groups + 1) * 32, BAR_STAGED + wg, BAR_DRAINED + wg, true};
    if constexpr (EW == 16) {
      if (groups == 2) {
        epilogue_loop<BN, INT8, ACT, OUTK, 256, true, EW, 2>(p, epi, acc_full, acc_empty, tmem_base, pair_id, num_pairs,
                                                             (int)rank * GEMM_BM, stage, warp);
      } else {
        epilogue_loop<BN, INT8, ACT, OUTK, 256, true, EW, 1>(p, epi, acc_full, acc_empty, tmem_base, pair_id, num_pairs,
                                                             (int)rank * GEMM_BM, stage, warp);
      }
    } else {
      epilogue_loop<BN, INT8, ACT, OUTK, 256, true, EW, 1>(p, epi, acc_full, acc_empty, tmem_base, pair_id, num_pairs,
                                                           (int)rank * GEMM_BM, stage, warp);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();                                   // the peer may still be reading this CTA's shared memory / barriers
  if (warp == W_MMA) ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
}

template <bool INT8, int ACT, int OUTK, int EW>
static hero_status launch_gemm_pair_ew(hero_handle* h, const CUtensorMap& tmA, const CUtensorMap& tmW, GemmParams p,
                                       cudaStream_t stream) {
  auto kern = gemm_pair_kernel<INT8, ACT, OUTK, EW>;
  // an 8-bit output of a short-K product leaves through a staging tile and bulk tensor stores when its base and row
  // pitch allow a tensor map; otherwise, and for wider outputs, every lane stores its own row
  CUtensorMap tmO;
  memset(&tmO, 0, sizeof(tmO));
  p.tma_out = 0;
  if constexpr (OUTK == OUT_I8 || OUTK == OUT_F8) {
    // worth it where the epilogue sets the pace: few k-blocks per tile (a long main loop hides the direct stores and
    // keeps all six pipeline stages)
    if (p.num_kb <= 16 && aligned16(p.out) && p.out_ld % 16 == 0) {
      hero_status st = make_tmap_2d(h, &tmO, p.out, 1, false, false, (uint64_t)p.M, (uint64_t)p.N, (uint64_t)p.out_ld, 128,
                                    GEMM_BM, 128);
      if (st != HERO_OK) return st;
      p.tma_out = 1;
    }
  }
  HERO_SMEM_OPT_IN(h, kern, PairCfg::SMEM_BYTES);
  const int tiles = p.num_m_tiles * p.num_n_tiles;
  const int pairs_max = h->sm_count / 2;
  const int pairs = tiles < pairs_max ? tiles : pairs_max;
  {
    LaunchScope scope(h, stream, KERNEL_GEMM);
    HERO_CUDA(launch_dependent(kern, dim3(2 * pairs), dim3((EW + 3) * 32), PairCfg::SMEM_BYTES, stream, tmA, tmW, tmO, p));
  }
  HERO_CUDA(cudaGetLastError());
  return HERO_OK;
}

// 16 epilogue warps when the epilogue sets the pace (an activation and few k-blocks per tile); 8 (with twice the
// registers and 32-column chunks) otherwise.
template <bool INT8, int ACT, int OUTK>
static hero_status launch_gemm_pair(hero_handle* h, const CUtensorMap& tmA, const CUtensorMap& tmW, const GemmParams& p,
                                    cudaStream_t stream) {
  if constexpr (OUTK != OUT_I32) {
    const bool wide_epi = ACT != HERO_ACT_NONE && p.num_kb <= 16;
    if (wide_epi) return launch_gemm_pair_ew<INT8, ACT, OUTK, 16>(h, tmA, tmW, p, stream);
  }
  return launch_gemm_pair_ew<INT8, ACT, OUTK, 8>(h, tmA, tmW, p, stream);
}

template <bool INT8>
static hero_status dispatch_epilogue_pair(hero_handle* h, const CUtensorMap& tmA, const CUtensorMap& tmW, const GemmParams& p,
                                          int act, cudaStream_t s) {
  if (p.out_dt == HERO_I32) {
    if constexpr (INT8) return launch_gemm_pair<true, HERO_ACT_NONE, OUT_I32>(h, tmA, tmW, p, s);
    else { set_error("raw INT32 output needs INT8 operands"); return HERO_ERR_UNSUPPORTED; }
  }
  if (p.out_dt == HERO_F8) {
    if constexpr (!INT8) {
      switch (act) {
        case HERO_ACT_NONE: return launch_gemm_pair<false, HERO_ACT_NONE, OUT_F8>(h, tmA, tmW, p, s);
        case HERO_ACT_GELU_ERF: return launch_gemm_pair<false, HERO_ACT_GELU_ERF, OUT_F8>(h, tmA, tmW, p, s);
        case HERO_ACT_GELU_TANH: return launch_gemm_pair<false, HERO_ACT_GELU_TANH, OUT_F8>(h, tmA, tmW, p, s);
      }
    }
    set_error("an e4m3 output needs e4m3 or FP operands");
    return HERO_ERR_UNSUPPORTED;
  }
  const bool i8 = p.out_dt == HERO_I8;
  switch (act) {
    case HERO_ACT_NONE:
      return i8 ? launch_gemm_pair<INT8, HERO_ACT_NONE, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm_pair<INT8, HERO_ACT_NONE, OUT_FP>(h, tmA, tmW, p, s);
    case HERO_ACT_GELU_ERF:
      return i8 ? launch_gemm_pair<INT8, HERO_ACT_GELU_ERF, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm_pair<INT8, HERO_ACT_GELU_ERF, OUT_FP>(h, tmA, tmW, p, s);
    case HERO_ACT_GELU_TANH:
      return i8 ? launch_gemm_pair<INT8, HERO_ACT_GELU_TANH, OUT_I8>(h, tmA, tmW, p, s)
                : launch_gemm_pair<INT8, HERO_ACT_GELU_TANH, OUT_FP>(h, tmA, tmW, p, s);
  }
  set_error("unknown activation %d", act);
  return HERO_ERR_INVALID_ARG;
}

static hero_status run_pair(hero_handle* h, const hero_linear_args* a, GemmParams& p, cudaStream_t s) {
  const bool int8 = a->A.dtype == HERO_I8, f8 = a->A.dtype == HERO_F8;
  const int eb = (int8 || f8) ? 1 : 2;
  const int kbox = GEMM_BK_BYTES / eb;
  p.num_m_tiles = (p.M + 255) / 256;
  p.num_n_tiles = (p.N + 255) / 256;
  const bool bf = a->A.dtype == HERO_BF16;
  p.idesc = int8 ? ptx::make_idesc(2, 1, 1, 0, 0, 256, 256)
                 : (f8 ? ptx::make_idesc(1, 0, 0, 0, 0, 256, 256) : ptx::make_idesc(1, bf ? 1 : 0, bf ? 1 : 0, 0, 0, 256, 256));
  CUtensorMap tmA, tmW;
  hero_status st = make_tmap_2d(h, &tmA, a->A.data, eb, a->A.dtype == HERO_F16, bf, (uint64_t)p.M, (uint64_t)p.K,
                                (uint64_t)a->A.ld * eb, kbox, GEMM_BM, 128);
  if (st != HERO_OK) return st;
  st = make_tmap_2d(h, &tmW, a->W, eb, a->A.dtype == HERO_F16, bf, (uint64_t)p.N, (uint64_t)p.K, (uint64_t)a->ldw * eb, kbox,
                    128, 128);
  if (st != HERO_OK) return st;
  if (int8) return dispatch_epilogue_pair<true>(h, tmA, tmW, p, a->act, s);
  return dispatch_epilogue_pair<false>(h, tmA, tmW, p, a->act, s);
}

template <int BN>
static hero_status run_bn(hero_handle* h, const hero_linear_args* a, GemmParams& p, cudaStream_t s) {
  const bool int8 = a->A.dtype == HERO_I8, f8 = a->A.dtype == HERO_F8;
  const int eb = (int8 || f8) ? 1 : 2;
  const int kbox = GEMM_BK_BYTES / eb;
  p.num_n_tiles = (p.N + BN - 1) / BN;
  p.idesc = int8 ? ptx::make_idesc(2, 1, 1, 0, 0, GEMM_BM, BN)
                 : (f8 ? ptx::make_idesc(1, 0, 0, 0, 0, GEMM_BM, BN)
                       : ptx::make_idesc(1, a->A.dtype == HERO_BF16 ? 1 : 0, a->A.dtype == HERO_BF16 ? 1 : 0, 0, 0, GEMM_BM, BN));
  CUtensorMap tmA, tmW;
  hero_status st = make_tmap_2d(h, &tmA, a->A.data, eb, a->A.dtype == HERO_F16, a->A.dtype == HERO_BF16, (uint64_t)p.M,
                                (uint64_t)p.K, (uint64_t)a->A.ld * eb, kbox, GEMM_BM, 128);
  if (st != HERO_OK) return st;
  st = make_tmap_2d(h, &tmW, a->W, eb, a->A.dtype == HERO_F16, a->A.dtype == HERO_BF16, (uint64_t)p.N, (uint64_t)p.K,
                    (uint64_t)a->ldw * eb, kbox, BN, 128);
  if (st != HERO_OK) return st;
  if (int8) return dispatch_epilogue<BN, true>(h, tmA, tmW, p, a->act, s);
  return dispatch_epilogue<BN, false>(h, tmA, tmW, p, a->act, s);
}


}  // namespace hero


extern "C" hero_status hero_w8a8_linear(hero_handle* h, const hero_linear_args* a, void* stream) {
  using namespace hero;
  HERO_REQUIRE(h && a, HERO_ERR_INVALID_ARG, "hero_w8a8_linear: NULL handle or args");
  hero_status st;
  if ((st = check_matrix(a->A, "A")) != HERO_OK) return st;
  if ((st = check_matrix(a->out, "out")) != HERO_OK) return st;
  const bool int8 = a->A.dtype == HERO_I8, f8 = a->A.dtype == HERO_F8, q8 = int8 || f8;
  HERO_REQUIRE(q8 || is_fp16ish(a->A.dtype), HERO_ERR_UNSUPPORTED, "A dtype %d: INT8, e4m3, F16 or BF16 expected", a->A.dtype);
  const int eb = q8 ? 1 : 2;
  HERO_REQUIRE(a->W != nullptr && aligned16(a->W), a->W ? HERO_ERR_ALIGNMENT : HERO_ERR_INVALID_ARG,
               "W must be a 16-byte aligned device pointer");
  HERO_REQUIRE(a->N > 0 && a->N % 16 == 0, HERO_ERR_UNSUPPORTED, "N=%lld must be a positive multiple of 16", (long long)a->N);
  const long long K = a->A.cols;
  HERO_REQUIRE((K * eb) % 16 == 0, HERO_ERR_UNSUPPORTED, "K=%lld: K * element size must be a multiple of 16 bytes", K);
  HERO_REQUIRE(a->ldw >= K && (a->ldw * eb) % 16 == 0, HERO_ERR_ALIGNMENT, "ldw=%lld invalid", (long long)a->ldw);
  HERO_REQUIRE(a->out.rows == a->A.rows && a->out.cols == a->N, HERO_ERR_INVALID_ARG, "out shape mismatch");
  HERO_REQUIRE(is_q8(a->out.dtype) || is_fp16ish(a->out.dtype) || a->out.dtype == HERO_I32, HERO_ERR_UNSUPPORTED,
               "out dtype %d", a->out.dtype);
  HERO_REQUIRE(a->out.dtype != HERO_F8 || !int8, HERO_ERR_UNSUPPORTED, "an e4m3 output needs e4m3 or FP operands");
  HERO_REQUIRE(a->out.dtype != HERO_I8 || !f8, HERO_ERR_UNSUPPORTED, "an INT8 output needs INT8 or FP operands");
  HERO_REQUIRE(!(is_q8(a->out.dtype) && a->out.gran == HERO_GRAN_TWQ), HERO_ERR_UNSUPPORTED,
               "a token-wise (TWQ) output needs a row reduction, which is kept out of GEMM epilogues (Sec. 2.1); "
               "fuse it into LN^quant instead");
  HERO_REQUIRE(a->out.dtype != HERO_I32 || int8, HERO_ERR_UNSUPPORTED, "raw INT32 output needs INT8 operands");
  if (q8) HERO_REQUIRE(a->w_scale != nullptr || a->out.dtype == HERO_I32, HERO_ERR_INVALID_ARG, "w_scale is required");
  HERO_REQUIRE(a->act >= HERO_ACT_NONE && a->act <= HERO_ACT_GELU_TANH, HERO_ERR_INVALID_ARG, "unknown activation %d", a->act);
  HERO_REQUIRE(a->A.rows < (1ll << 31) && a->N < (1ll << 31) && K < (1ll << 31), HERO_ERR_UNSUPPORTED, "dimension too large");
  HERO_REQUIRE(a->out_col_absmax == nullptr || is_fp16ish(a->out.dtype), HERO_ERR_UNSUPPORTED,
               "out_col_absmax observes an F16 / BF16 output (calibration runs the modules in FP mode)");
  if (a->A.rows == 0) return HERO_OK;

  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = (int)a->A.rows; p.N = (int)a->N; p.K = (int)K;
  p.num_m_tiles = (p.M + GEMM_BM - 1) / GEMM_BM;
  p.num_kb = (int)((K * eb + GEMM_BK_BYTES - 1) / GEMM_BK_BYTES);
  p.rs = (q8 && a->A.gran == HERO_GRAN_TWQ) ? a->A.scale : nullptr;
  p.cs = q8 ? a->w_scale : nullptr;
  p.f8 = f8 ? 1 : 0;
  p.bias = a->bias; p.post = a->post_scale;
  p.out = a->out.data; p.out_ld = a->out.ld; p.out_dt = a->out.dtype;
  p.elem_bytes = eb;
  p.obs_col = a->out_col_absmax;
  p.err = h->d_error;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Few rows: streaming W bounds the time.  The tile kernels below give one row-tile N / 64 CTAs at most, each walking
  // the whole K; the few-row kernel splits K over a cluster instead.  It wins whenever M <= 16, and for wider inputs
  // when the tile kernels would leave SMs idle on a long K (measured on the M in {16..128} x K, N in {1024..16384} grid).
  if (p.M <= GEMM_BM && p.obs_col == nullptr) {            // (the few-row kernel has no observer)
    const bool idle = (p.N + 63) / 64 < h->sm_count;
    const long long kbytes = K * eb;
    if (p.M <= 16 || (idle && kbytes >= 8192) || (idle && kbytes >= 4096 && p.M <= 32)) return run_skinny(h, a, p, s);
  }
  // widest column tile that still gives every SM a tile
  const long long t256 = (long long)p.num_m_tiles * ((p.N + 255) / 256);
  const long long t128 = (long long)p.num_m_tiles * ((p.N + 127) / 128);
  const long long enough = (long long)h->sm_count * 6 / 10;
  const long long tpair = (long long)((p.M + 255) / 256) * ((p.N + 255) / 256);
  if (tpair * 2 >= enough && p.M > GEMM_BM) return run_pair(h, a, p, s);
  if (t256 >= enough) return run_bn<256>(h, a, p, s);
  if (t128 >= enough) return run_bn<128>(h, a, p, s);
  return run_bn<64>(h, a, p, s);
}

