// Small entry points that belong to no kernel: error strings and the version.
#include "common.cuh"

extern "C" const char* slicemoe_strerror(int code) {
  switch (code) {
    case SLICEMOE_OK: return "ok";
    case SLICEMOE_E_INVALID_ARG: return "invalid argument";
    case SLICEMOE_E_UNSUPPORTED: return "unsupported format or size";
    case SLICEMOE_E_CUDA: return "CUDA runtime error";
    case SLICEMOE_E_NOMEM: return "host allocation failed";
    default: return "unknown error code";
  }
}

extern "C" int slicemoe_version(void) { return 100; }

int g_slicemoe_last_cuda_error = 0;

extern "C" const char* slicemoe_last_cuda_error(void) {
  return cudaGetErrorString((cudaError_t)g_slicemoe_last_cuda_error);
}
