// Handle life cycle, error text, tensor-map construction, Table 1 presets.
#include <mutex>
#include <unordered_set>
#include "common.cuh"

namespace hero {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

// streams on which a library call has just written model constants (see launch_dependent)
static std::mutex g_fence_mutex;
static std::unordered_set<cudaStream_t> g_fenced;
void pdl_fence_stream(cudaStream_t s) {
  std::lock_guard<std::mutex> lock(g_fence_mutex);
  g_fenced.insert(s);
}
bool pdl_take_fence(cudaStream_t s) {
  std::lock_guard<std::mutex> lock(g_fence_mutex);
  return g_fenced.erase(s) != 0;
}

hero_status cuda_fail(cudaError_t e, const char* what) {
  set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
  return HERO_ERR_CUDA;
}

hero_status check_matrix(const hero_tensor& t, const char* name) {
  size_t es = dtype_size(t.dtype);
  HERO_REQUIRE(es != 0, HERO_ERR_INVALID_ARG, "%s: unknown dtype %d", name, t.dtype);
  HERO_REQUIRE(t.data != nullptr || t.rows == 0, HERO_ERR_INVALID_ARG, "%s: data is NULL", name);
  HERO_REQUIRE(t.rows >= 0 && t.cols > 0 && t.ld >= t.cols, HERO_ERR_INVALID_ARG,
               "%s: bad shape rows=%lld cols=%lld ld=%lld", name, (long long)t.rows, (long long)t.cols,
               (long long)t.ld);
  HERO_REQUIRE(aligned16(t.data), HERO_ERR_ALIGNMENT, "%s: data pointer is not 16-byte aligned", name);
  HERO_REQUIRE((t.ld * es) % 16 == 0, HERO_ERR_ALIGNMENT, "%s: row pitch %lld bytes is not a multiple of 16", name,
               (long long)(t.ld * es));
  if (is_q8(t.dtype) && t.gran != HERO_GRAN_NONE)
    HERO_REQUIRE(t.scale != nullptr, HERO_ERR_INVALID_ARG, "%s: 8-bit tensor with granularity %d needs a scale", name,
                 t.gran);
  return HERO_OK;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

hero_status make_tmap_2d(const hero_handle* h, CUtensorMap* out, const void* base, int elem_bytes, bool is_fp16,
                         bool is_bf16, uint64_t rows, uint64_t cols, uint64_t ld_bytes, uint32_t box_cols,
                         uint32_t box_rows, int swizzle_bytes) {
  HERO_REQUIRE(h && h->encode_tiled, HERO_ERR_CUDA, "tensor-map encoder unavailable");
  // cache look-up (see hero_tmap_slot)
  const uint64_t key[5] = {reinterpret_cast<uint64_t>(base), rows, cols, ld_bytes,
                           (uint64_t)box_cols | ((uint64_t)box_rows << 16) | ((uint64_t)elem_bytes << 32) |
                               ((uint64_t)(is_bf16 ? 1 : 0) << 40) | ((uint64_t)swizzle_bytes << 44)};
  uint64_t hsh = 0x9E3779B97F4A7C15ull;
  for (int i = 0; i < 5; ++i) hsh = (hsh ^ key[i]) * 0xBF58476D1CE4E5B9ull + (hsh >> 29);
  hero_handle* hm = const_cast<hero_handle*>(h);
  hero_tmap_slot& slot = hm->tmap[(hsh >> 32) % HERO_TMAP_SLOTS];
  std::lock_guard<std::mutex> guard(hm->tmap_mu);
  if (slot.used && memcmp(slot.key, key, sizeof(key)) == 0) {
    *out = slot.map;
    return HERO_OK;
  }
  CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_UINT8;
  if (elem_bytes == 2) dt = is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
  (void)is_fp16;
  CUtensorMapSwizzle sw = CU_TENSOR_MAP_SWIZZLE_NONE;
  if (swizzle_bytes == 32) sw = CU_TENSOR_MAP_SWIZZLE_32B;
  if (swizzle_bytes == 64) sw = CU_TENSOR_MAP_SWIZZLE_64B;
  if (swizzle_bytes == 128) sw = CU_TENSOR_MAP_SWIZZLE_128B;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<encode_tiled_fn>(h->encode_tiled)(
      out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  HERO_REQUIRE(r == CUDA_SUCCESS, HERO_ERR_CUDA,
               "cuTensorMapEncodeTiled failed (%d): rows=%llu cols=%llu ld_bytes=%llu box=%ux%u", (int)r,
               (unsigned long long)rows, (unsigned long long)cols, (unsigned long long)ld_bytes, box_cols, box_rows);
  memcpy(slot.key, key, sizeof(key));
  slot.map = *out;
  slot.used = true;
  return HERO_OK;
}

}  // namespace hero

extern "C" {

const char* hero_last_error(void) { return hero::g_err; }

hero_status hero_create(hero_handle** out) {
  HERO_REQUIRE(out != nullptr, HERO_ERR_INVALID_ARG, "hero_create: out is NULL");
  *out = nullptr;
  int dev = 0;
  HERO_CUDA(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  HERO_CUDA(cudaGetDeviceProperties(&prop, dev));
  HERO_REQUIRE(prop.major == 10, HERO_ERR_UNSUPPORTED,
               "this library is built for sm_100a only; device %d is sm_%d%d", dev, prop.major, prop.minor);
  hero_handle* h = new hero_handle();
  h->device = dev;
  h->sm_count = prop.multiProcessorCount;
  h->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
  h->launches.store(0);
  h->d_error = nullptr;
  h->encode_tiled = nullptr;
  h->prof_on = false; h->prof_cap = 0; h->prof_n = 0; h->prof_ev = nullptr; h->prof_tag = nullptr;
  cudaError_t e = cudaMalloc(&h->d_error, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(h->d_error, 0, sizeof(int));
  if (e != cudaSuccess) {
    delete h;
    return hero::cuda_fail(e, "allocating the device error word");
  }
  cudaDriverEntryPointQueryResult qres;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &h->encode_tiled, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !h->encode_tiled) {
    cudaFree(h->d_error);
    delete h;
    hero::set_error("cuTensorMapEncodeTiled could not be resolved");
    return HERO_ERR_CUDA;
  }
  *out = h;
  return HERO_OK;
}

static void free_profile(hero_handle* h) {
  for (int i = 0; i < 2 * h->prof_cap; ++i) cudaEventDestroy(h->prof_ev[i]);
  delete[] h->prof_ev; delete[] h->prof_tag;
  h->prof_ev = nullptr; h->prof_tag = nullptr; h->prof_cap = 0; h->prof_n = 0; h->prof_on = false;
}

hero_status hero_profile_begin(hero_handle* h, int32_t max_launches) {
  HERO_REQUIRE(h != nullptr && max_launches > 0, HERO_ERR_INVALID_ARG, "hero_profile_begin: bad arguments");
  if (h->prof_cap != max_launches) {
    free_profile(h);
    h->prof_ev = new cudaEvent_t[2 * max_launches];
    h->prof_tag = new int32_t[max_launches];
    for (int i = 0; i < 2 * max_launches; ++i) HERO_CUDA(cudaEventCreate(&h->prof_ev[i]));
    h->prof_cap = max_launches;
  }
  h->prof_n = 0;
  h->prof_on = true;
  return HERO_OK;
}

hero_status hero_profile_end(hero_handle* h, float* ms_out, int32_t* tag_out, int32_t* n_out) {
  HERO_REQUIRE(h != nullptr && n_out != nullptr, HERO_ERR_INVALID_ARG, "hero_profile_end: bad arguments");
  h->prof_on = false;
  for (int i = 0; i < h->prof_n; ++i) {
    HERO_CUDA(cudaEventSynchronize(h->prof_ev[2 * i + 1]));
    float ms = 0.f;
    HERO_CUDA(cudaEventElapsedTime(&ms, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]));
    if (ms_out) ms_out[i] = ms;
    if (tag_out) tag_out[i] = h->prof_tag[i];
  }
  *n_out = h->prof_n;
  return HERO_OK;
}

hero_status hero_destroy(hero_handle* h) {
  if (!h) return HERO_OK;
  free_profile(h);
  cudaFree(h->d_error);
  delete h;
  return HERO_OK;
}

hero_status hero_check(hero_handle* h, void* stream) {
  HERO_REQUIRE(h != nullptr, HERO_ERR_INVALID_ARG, "hero_check: handle is NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  HERO_CUDA(cudaStreamSynchronize(s));
  int code = 0;
  HERO_CUDA(cudaMemcpy(&code, h->d_error, sizeof(int), cudaMemcpyDeviceToHost));
  if (code != 0) {
    cudaMemset(h->d_error, 0, sizeof(int));
    if (code == hero::ERR_BAD_ID) {
      hero::set_error("an embedding id was outside its table; it was clamped to the nearest valid row");
      return HERO_ERR_INVALID_ARG;
    }
    hero::set_error("a bounded device-side wait gave up (code 0x%x)", code);
    return HERO_ERR_DEVICE_TIMEOUT;
  }
  return HERO_OK;
}

int64_t hero_launch_count(const hero_handle* h) { return h ? h->launches.load(std::memory_order_relaxed) : 0; }

hero_status hero_mode_preset(int32_t preset, int32_t mode_out[5]) {
  HERO_REQUIRE(mode_out != nullptr, HERO_ERR_INVALID_ARG, "hero_mode_preset: mode_out is NULL");
  // Table 1 columns: QKV GeMM, Attn., Attn. Output, FC1, FC2 (Embedding is INT8 in M1-M3).
  static const int32_t table[4][5] = {
      {HERO_MODE_FP, HERO_MODE_FP, HERO_MODE_FP, HERO_MODE_FP, HERO_MODE_FP},          // all FP
      {HERO_MODE_INT8, HERO_MODE_FP, HERO_MODE_FP, HERO_MODE_INT8, HERO_MODE_FP},      // M1
      {HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_FP},  // M2
      {HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_INT8, HERO_MODE_INT8} // M3
  };
  HERO_REQUIRE(preset >= 0 && preset <= 3, HERO_ERR_INVALID_ARG, "unknown preset %d", preset);
  for (int i = 0; i < 5; ++i) mode_out[i] = table[preset][i];
  return HERO_OK;
}

}  // extern "C"
