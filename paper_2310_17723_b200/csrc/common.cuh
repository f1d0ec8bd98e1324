// Shared host-side plumbing of the library: the handle, error reporting, argument checks.
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <cstdarg>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>

#include "../../include/hero.h"
#ifdef __CUDACC__
#include <cuda_fp16.h>
#endif

// A tensor map is a pure function of (base, shape, pitch, box, type, swizzle); encoding one costs about a microsecond of
// host time, several per launch.  Layers launch the same shapes on the same buffers over and over: a small direct-mapped
// cache in the handle spares the latency-bound workloads that host time.
struct hero_tmap_slot {
  uint64_t key[5];
  CUtensorMap map;
  bool used = false;
};
constexpr int HERO_TMAP_SLOTS = 128;

struct hero_handle {
  int device;
  int sm_count;
  int max_smem_optin;
  int* d_error;        // device error word: 0 = fine, else a code saying which wait gave up
  std::atomic<int64_t> launches;   // bumped by every launch; several host threads may share a handle's counter
  void* encode_tiled;  // cuTensorMapEncodeTiled, resolved through the runtime
  // optional per-launch timing (hero_profile_begin / _end): event pairs around every kernel launch
  bool prof_on;
  int prof_cap, prof_n;
  cudaEvent_t* prof_ev;   // 2 * prof_cap events
  int32_t* prof_tag;      // kernel family of each recorded launch
  std::mutex tmap_mu;     // several host threads may share a handle
  hero_tmap_slot tmap[HERO_TMAP_SLOTS];
};

namespace hero {

void set_error(const char* fmt, ...);
hero_status cuda_fail(cudaError_t e, const char* what);

#define HERO_CUDA(call)                                   \
  do {                                                    \
    cudaError_t _e = (call);                              \
    if (_e != cudaSuccess) return hero::cuda_fail(_e, #call); \
  } while (0)

#define HERO_REQUIRE(cond, status, ...)  \
  do {                                   \
    if (!(cond)) {                       \
      hero::set_error(__VA_ARGS__);      \
      return (status);                   \
    }                                    \
  } while (0)

inline size_t dtype_size(int dt) {
  switch (dt) {
    case HERO_I8: case HERO_U8: case HERO_F8: return 1;
    case HERO_F16: case HERO_BF16: return 2;
    case HERO_I32: case HERO_F32: return 4;
    default: return 0;
  }
}
inline bool is_fp16ish(int dt) { return dt == HERO_F16 || dt == HERO_BF16; }
#ifdef __CUDACC__
__host__ __device__
#endif
inline bool is_q8(int dt) { return dt == HERO_I8 || dt == HERO_F8; }   // 8-bit payload that carries a scale
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// data pointer 16-byte aligned, row pitch a multiple of 16 bytes, ld >= cols
hero_status check_matrix(const hero_tensor& t, const char* name);

// Codes a kernel may leave in the device error word besides "a bounded wait gave up" (those carry the place in
// their low 16 bits and nothing above): an embedding id outside its table, clamped by LN^quant's gather.
constexpr int ERR_BAD_ID = 0x1D000001;

// Kernel families for the per-launch timing records.
enum { KERNEL_LN = 1, KERNEL_GEMM = 2, KERNEL_ATTN = 3 };
// Brackets one kernel launch with events when timing is on; counts the launch either way.
struct LaunchScope {
  hero_handle* h; cudaStream_t s; int slot;
  LaunchScope(hero_handle* h_, cudaStream_t s_, int tag) : h(h_), s(s_), slot(-1) {
    h->launches.fetch_add(1, std::memory_order_relaxed);
    if (h->prof_on && h->prof_n < h->prof_cap) {
      slot = h->prof_n++;
      h->prof_tag[slot] = tag;
      cudaEventRecord(h->prof_ev[2 * slot], s);
    }
  }
  ~LaunchScope() { if (slot >= 0) cudaEventRecord(h->prof_ev[2 * slot + 1], s); }
};

// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) and occupancy figures belong to a
// (kernel, device) pair, not to the process.  One of these per kernel instantiation (a function-local static)
// remembers per device ordinal what has been set; lock-free, and a lost race only repeats an idempotent call.
constexpr int MAX_DEVICES = 64;
struct PerDeviceOnce {
  std::atomic<uint64_t> mask{0};
  bool done(int dev) const { return dev >= 0 && dev < MAX_DEVICES && ((mask.load(std::memory_order_acquire) >> dev) & 1); }
  void set(int dev) { if (dev >= 0 && dev < MAX_DEVICES) mask.fetch_or(1ull << dev, std::memory_order_release); }
};
struct PerDeviceInt {
  std::atomic<int> v[MAX_DEVICES];
  PerDeviceInt() { for (auto& x : v) x.store(0, std::memory_order_relaxed); }
  int get(int dev) const { return dev >= 0 && dev < MAX_DEVICES ? v[dev].load(std::memory_order_acquire) : 0; }
  void set(int dev, int x) { if (dev >= 0 && dev < MAX_DEVICES) v[dev].store(x, std::memory_order_release); }
};
// Opts `kern` in to `bytes` of dynamic shared memory on the handle's device, once per device.
#define HERO_SMEM_OPT_IN(h, kern, bytes)                                                                 \
  do {                                                                                                   \
    static hero::PerDeviceOnce _once;                                                                    \
    if (!_once.done((h)->device)) {                                                                      \
      HERO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes))); \
      _once.set((h)->device);                                                                            \
    }                                                                                                    \
  } while (0)

// Kernel launch with programmatic dependent launch allowed: the grid may be scheduled while the previous kernel of
// the stream is still draining, runs its set-up (barrier init, tensor-memory allocation, descriptor prefetch) and then
// blocks in griddepcontrol.wait until that kernel has completed and its writes are visible.  Every kernel of the
// library executes griddepcontrol.launch_dependents first thing and griddepcontrol.wait before its first global
// memory access, so launch latency and ramp-up overlap the predecessor's tail and nothing else changes.
//
// Model constants (weight matrices) may be fetched BEFORE the dependency wait: they are not produced by the layer's own
// kernels.  A library call that writes such constants on a stream (hero_quantize_weight) therefore fences the stream:
// the next launch on it is an ordinary, fully serialised one, and with it everything launched after.
void pdl_fence_stream(cudaStream_t s);     // the next launch on `s` must not start before earlier work has completed
bool pdl_take_fence(cudaStream_t s);       // true once after pdl_fence_stream(s)

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_take_fence(s) ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

#ifdef __CUDACC__
namespace ptx {
// e4m3 <-> FP32 through the conversion instructions: two values per instruction
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {   // saturating, round to nearest even
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t f32x4_to_e4m3x4(float a, float b, float c, float d) {
  return f32x2_to_e4m3x2(a, b) | (f32x2_to_e4m3x2(c, d) << 16);
}
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t two) {          // low byte -> .x
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)two));
  const __half2 h = *reinterpret_cast<const __half2*>(&h2);
  return __half22float2(h);
}
// launch_dependents: the next kernel of the stream may start being scheduled.  wait: returns once the previous kernel
// of the stream has completed and flushed its writes (immediately if there is none or the launch was an ordinary one).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
}  // namespace ptx
#endif

// 2-D TMA descriptor over a row-major matrix [rows, cols] of `elem_bytes` elements with row pitch
// ld_bytes; box = box_cols x box_rows elements; swizzle_bytes in {0, 32, 64, 128}.
hero_status make_tmap_2d(const hero_handle* h, CUtensorMap* out, const void* base, int elem_bytes, bool is_fp16,
                         bool is_bf16, uint64_t rows, uint64_t cols, uint64_t ld_bytes, uint32_t box_cols,
                         uint32_t box_rows, int swizzle_bytes);

}  // namespace hero
