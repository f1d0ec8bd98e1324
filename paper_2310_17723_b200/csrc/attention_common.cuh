// Pieces shared by the INT8 and the FP16/BF16 attention kernels: launch constants, parameters, tile walk.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include <climits>
#include <cmath>
#include <cuda_fp16.h>
#include <cuda_bf16.h>

namespace hero {

constexpr int ATT_BM = 128;      // queries per CTA
constexpr int ATT_BN = 128;      // keys per block
constexpr int ATT_THREADS = 576;
constexpr int ATT_SM_WARPS = 16;       // softmax warps
constexpr int ATT_NSB = 3;             // score buffers in tensor memory (3 x 128 columns + dh output columns = 512)
constexpr int ATT_TMA_WARP = 16, ATT_MMA_WARP = 17;
constexpr float ATT_MAGIC = 12582912.0f; // 1.5 * 2^23

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
  float* p_absmax;         // calibration observer of the FP core: running max of the softmax probabilities, or NULL
  float* obs_col;          // calibration observer of the FP core: per-column running absmax of an FP output, or NULL
  // verification outputs (hero_int8_attention_probe; kernels compiled with PROBE only): raw Q K^T accumulators and
  // P codes [B*nh][S][S], raw P V accumulators [B*S][nh*dh]; each may be NULL
  int* dbg_scores;
  uint8_t* dbg_p;
  int* dbg_acc;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// exact float of an INT32 score with |a| < 2^22 (|a| <= 127^2 * 128), without the conversion unit
__device__ __forceinline__ float score_to_float(uint32_t a) { return __uint_as_float(0x4B400000u + a) - ATT_MAGIC; }
__device__ __forceinline__ uint32_t low_bytes4_u(float a, float b, float c, float d) {
  const uint32_t ab = __byte_perm(__float_as_uint(a), __float_as_uint(b), 0x0040);
  const uint32_t cd = __byte_perm(__float_as_uint(c), __float_as_uint(d), 0x0040);
  return __byte_perm(ab, cd, 0x5410);
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

// Tile t of the persistent loop -> (query tile, head, batch).  Late query tiles first: under a causal mask
// they carry the most key blocks, so the work a CTA picks up shrinks towards the end of the kernel.
__device__ __forceinline__ void attn_tile(const AttnParams& p, int t, int& qt, int& h, int& b) {
  const int bh = p.B * p.nh;
  qt = p.nqt - 1 - t / bh;
  const int r = t % bh;
  h = r % p.nh;
  b = r / p.nh;
}
__device__ __forceinline__ int attn_nkv(const AttnParams& p, int qt, int b, int& klen) {
  klen = p.S;
  if (p.key_len) klen = min(p.S, max(0, p.key_len[b]));
  int kv_end = klen;
  if (p.mask == HERO_MASK_CAUSAL) kv_end = min(kv_end, qt * ATT_BM + ATT_BM);
  return (kv_end + ATT_BN - 1) / ATT_BN;
}


// FP16 / BF16 attention for a module left in FP mode (Table 1); defined in attention_fp.cu
hero_status attn_fp_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream);
// INT8 core with the whole score row resident in tensor memory (S <= 512); defined in attention_resident.cu
hero_status attn_resident_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream, bool probe);
// INT8 core for S <= 512 as a pipeline of exponential and pack warps; defined in attention_pipe.cu
hero_status attn_pipe_dispatch(hero_handle* h, const hero_attn_args* a, AttnParams& p, cudaStream_t stream, bool probe);

// A position in a ring of N slots with the phase parity of its barriers, advanced without divisions (the ring depths here are not powers of two).
template <int N>
struct RingPos {
  int idx = 0;
  uint32_t par = 0;
  __device__ __forceinline__ void advance(int n) {          // n <= 2 N
    idx += n;
    if (idx >= N) { idx -= N; par ^= 1; }
    if (idx >= N) { idx -= N; par ^= 1; }
  }
  // slot and parity k positions further on (k <= N)
  __device__ __forceinline__ void at(int k, int& slot, uint32_t& parity) const {
    slot = idx + k; parity = par;
    if (slot >= N) { slot -= N; parity ^= 1; }
  }
};


}  // namespace hero
