// hero_layer_forward_static: the layer forward for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code that runs inside another framework's
// memory plan (every byte of the device is already handed out and accounted for), plugin or real-time paths
// where an allocation could block on the driver or fail late, and processes that are only given the buffers
// they were started with.  hero_layer_forward needs a workspace from its caller and a handle whose creation
// allocates; this entry point needs neither.  Its scratch is a fixed array that is part of the loaded library
// image, so every GPU that loads libhero.so carries it until the process exits.
#include "common.cuh"

#include <mutex>

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = 64ull << 20;     // 64 MiB: the largest layer workspace this entry point serves

// File-scope device storage.  In host code these names are only host-side stand-ins, not device addresses:
// the real addresses are fetched once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];
static __device__ int g_static_error_word;

struct StaticState {
  bool ready = false;
  hero_handle handle;
  void* scratch = nullptr;
};
StaticState g_state[hero::MAX_DEVICES];
std::mutex g_mutex;

// One-time set-up for the current device: no allocation, only queries and symbol look-ups.
hero_status setup_device(int dev, StaticState** out) {
  std::lock_guard<std::mutex> lock(g_mutex);
  StaticState& s = g_state[dev];
  if (!s.ready) {
    cudaDeviceProp prop;
    HERO_CUDA(cudaGetDeviceProperties(&prop, dev));
    HERO_REQUIRE(prop.major == 10, HERO_ERR_UNSUPPORTED, "this library is built for sm_100a only; device %d is sm_%d%d", dev,
                 prop.major, prop.minor);
    void* scratch = nullptr;
    void* err_word = nullptr;
    HERO_CUDA(cudaGetSymbolAddress(&scratch, g_static_scratch));
    HERO_CUDA(cudaGetSymbolAddress(&err_word, g_static_error_word));
    HERO_REQUIRE(scratch != nullptr && err_word != nullptr, HERO_ERR_CUDA, "static scratch has no device address");
    void* encode = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &encode, cudaEnableDefault, &qres);
    HERO_REQUIRE(e == cudaSuccess && qres == cudaDriverEntryPointSuccess && encode != nullptr, HERO_ERR_CUDA,
                 "cuTensorMapEncodeTiled could not be resolved");
    s.handle.launches.store(0);
    s.handle.prof_on = false; s.handle.prof_cap = 0; s.handle.prof_n = 0;
    s.handle.prof_ev = nullptr; s.handle.prof_tag = nullptr;
    s.handle.device = dev;
    s.handle.sm_count = prop.multiProcessorCount;
    s.handle.max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    s.handle.d_error = static_cast<int*>(err_word);
    s.handle.encode_tiled = encode;
    s.scratch = scratch;
    s.ready = true;
  }
  *out = &s;
  return HERO_OK;
}

}  // namespace

extern "C" hero_status hero_layer_workspace_bytes(const hero_layer_desc* d, int64_t M, size_t* bytes);
extern "C" hero_status hero_layer_forward(hero_handle* h, const hero_layer_desc* d, const hero_tensor* in,
                                          const hero_tensor* pending, const hero_tensor* out, void* workspace,
                                          size_t workspace_bytes, void* stream);

extern "C" hero_status hero_layer_forward_static(const hero_layer_desc* d, const hero_tensor* in, const hero_tensor* pending,
                                                 const hero_tensor* out, void* stream) {
  HERO_REQUIRE(d && in && out, HERO_ERR_INVALID_ARG, "hero_layer_forward_static: NULL argument");
  size_t need = 0;
  hero_status st = hero_layer_workspace_bytes(d, in->rows, &need);
  if (st != HERO_OK) return st;
  HERO_REQUIRE(need <= STATIC_SCRATCH_BYTES, HERO_ERR_WORKSPACE,
               "this layer needs %zu bytes of scratch; the built-in scratch of hero_layer_forward_static holds %zu "
               "(use hero_layer_forward with a caller-provided workspace for larger layers)",
               need, STATIC_SCRATCH_BYTES);
  int dev = 0;
  HERO_CUDA(cudaGetDevice(&dev));
  HERO_REQUIRE(dev >= 0 && dev < hero::MAX_DEVICES, HERO_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  StaticState* s = nullptr;
  if ((st = setup_device(dev, &s)) != HERO_OK) return st;
  // Every intermediate the layer reads is written by an earlier kernel of the same call, so nothing in the
  // scratch has to start at zero; what a previous call left there is simply overwritten.
  return hero_layer_forward(&s->handle, d, in, pending, out, s->scratch, STATIC_SCRATCH_BYTES, stream);
}

// The device error word of hero_layer_forward_static (the entry point has no handle for hero_check to look at).
// Synchronizes `stream`, copies the word back with a symbol copy (no allocation), clears it and reports what it held.
extern "C" hero_status hero_static_check(void* stream) {
  HERO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  int code = 0;
  HERO_CUDA(cudaMemcpyFromSymbol(&code, g_static_error_word, sizeof(int)));
  if (code == 0) return HERO_OK;
  const int zero = 0;
  HERO_CUDA(cudaMemcpyToSymbol(g_static_error_word, &zero, sizeof(int)));
  if (code == hero::ERR_BAD_ID) {
    hero::set_error("an embedding id was outside its table; it was clamped to the nearest valid row");
    return HERO_ERR_INVALID_ARG;
  }
  hero::set_error("a bounded device-side wait gave up (code 0x%x)", code);
  return HERO_ERR_DEVICE_TIMEOUT;
}
