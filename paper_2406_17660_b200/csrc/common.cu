// Status word, status strings and grass_device_status.
#include "common.cuh"

namespace grass {

// One status word per device that loads the library: [0] code, [1] detail.
__device__ int g_status_word[4];

int* status_word(cudaError_t* err) {
  static int* cached[64] = {nullptr};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_status_word);
    if (*err != cudaSuccess) return nullptr;
    cached[dev] = static_cast<int*>(p);
  }
  return cached[dev];
}

namespace {
struct Profile {
  bool active = false;
  int cap = 0, seen = 0;
  cudaEvent_t* start = nullptr;
  cudaEvent_t* stop = nullptr;
  int* kid = nullptr;
} g_profile;
}  // namespace

void profile_mark_begin(int kernel_id, cudaStream_t s) {
  if (!g_profile.active) return;
  if (g_profile.seen < g_profile.cap) {
    g_profile.kid[g_profile.seen] = kernel_id;
    cudaEventRecord(g_profile.start[g_profile.seen], s);
  }
}
void profile_mark_end(cudaStream_t s) {
  if (!g_profile.active) return;
  if (g_profile.seen < g_profile.cap) cudaEventRecord(g_profile.stop[g_profile.seen], s);
  ++g_profile.seen;
}

}  // namespace grass

extern "C" int grass_profile_begin(int32_t max_launches) {
  using grass::g_profile;
  if (max_launches < 1 || g_profile.active) return GRASS_ERR_INVALID_ARG;
  g_profile.start = new cudaEvent_t[max_launches];
  g_profile.stop = new cudaEvent_t[max_launches];
  g_profile.kid = new int[max_launches];
  for (int i = 0; i < max_launches; ++i) {
    GRASS_CUDA_TRY(cudaEventCreate(&g_profile.start[i]));
    GRASS_CUDA_TRY(cudaEventCreate(&g_profile.stop[i]));
  }
  g_profile.cap = max_launches;
  g_profile.seen = 0;
  g_profile.active = true;
  return GRASS_OK;
}

extern "C" int grass_profile_end_timeline(int32_t* kernel_id, float* ms, float* start_ms,
                                          int32_t* n_launches);

extern "C" int grass_profile_end(int32_t* kernel_id, float* ms, int32_t* n_launches) {
  return grass_profile_end_timeline(kernel_id, ms, nullptr, n_launches);
}

extern "C" int grass_profile_end_timeline(int32_t* kernel_id, float* ms, float* start_ms,
                                          int32_t* n_launches) {
  using grass::g_profile;
  if (!g_profile.active) return GRASS_ERR_INVALID_ARG;
  g_profile.active = false;
  int rc = GRASS_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) rc = GRASS_ERR_CUDA;
  const int timed = g_profile.seen < g_profile.cap ? g_profile.seen : g_profile.cap;
  for (int i = 0; i < timed && rc == GRASS_OK; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_profile.start[i], g_profile.stop[i]) != cudaSuccess)
      rc = GRASS_ERR_CUDA;
    if (ms != nullptr) ms[i] = t;
    if (kernel_id != nullptr) kernel_id[i] = g_profile.kid[i];
    if (start_ms != nullptr &&
        cudaEventElapsedTime(&start_ms[i], g_profile.start[0], g_profile.start[i]) != cudaSuccess)
      rc = GRASS_ERR_CUDA;
  }
  if (n_launches != nullptr) *n_launches = g_profile.seen;
  for (int i = 0; i < g_profile.cap; ++i) {
    cudaEventDestroy(g_profile.start[i]);
    cudaEventDestroy(g_profile.stop[i]);
  }
  delete[] g_profile.start;
  delete[] g_profile.stop;
  delete[] g_profile.kid;
  g_profile.start = g_profile.stop = nullptr;
  g_profile.kid = nullptr;
  g_profile.cap = g_profile.seen = 0;
  return rc;
}

extern "C" int grass_device_status(void* stream, int32_t* detail) {
  cudaError_t err;
  int* word = grass::status_word(&err);
  if (word == nullptr) {
    fprintf(stderr, "grass: status word unavailable: %s\n", cudaGetErrorString(err));
    return GRASS_ERR_CUDA;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int host[2] = {0, 0};
  GRASS_CUDA_TRY(cudaMemcpyAsync(host, word, sizeof(host), cudaMemcpyDeviceToHost, s));
  GRASS_CUDA_TRY(cudaMemsetAsync(word, 0, 4 * sizeof(int), s));
  GRASS_CUDA_TRY(cudaStreamSynchronize(s));
  if (detail != nullptr) *detail = host[1];
  return host[0];
}

extern "C" const char* grass_status_string(int status) {
  switch (status) {
    case GRASS_OK: return "ok";
    case GRASS_ERR_INVALID_ARG: return "invalid argument";
    case GRASS_ERR_ALIGNMENT: return "pointer or pitch not aligned for this path";
    case GRASS_ERR_UNSUPPORTED: return "unsupported dtype or method";
    case GRASS_ERR_DEGENERATE: return "degenerate row norms";
    case GRASS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GRASS_ERR_CUDA: return "CUDA call failed";
    case GRASS_ERR_TIMEOUT: return "device-side wait ran out";
    default: return "unknown status";
  }
}
