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

}  // namespace grass

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
