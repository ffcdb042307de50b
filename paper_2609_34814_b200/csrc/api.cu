// Status strings, thread-local error text, device queries.
#include "host_common.h"

namespace waveal {
static thread_local char g_err[512] = "";
static thread_local int32_t g_launches = 0;
char* last_error_buffer() { return g_err; }
int32_t& launch_counter() { return g_launches; }
}  // namespace waveal

extern "C" const char* waveal_status_string(waveal_status s) {
  switch (s) {
    case WAVEAL_OK: return "ok";
    case WAVEAL_ERR_INVALID_ARG: return "invalid argument";
    case WAVEAL_ERR_UNSUPPORTED: return "unsupported configuration";
    case WAVEAL_ERR_WORKSPACE: return "workspace missing or too small";
    case WAVEAL_ERR_BAD_MASK: return "bad mask (device-side check)";
    case WAVEAL_ERR_CUDA: return "CUDA call failed";
    case WAVEAL_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" const char* waveal_last_error(void) { return waveal::g_err; }

extern "C" int32_t waveal_last_launch_count(void) { return waveal::g_launches; }

extern "C" int32_t waveal_default_wave_size(void) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
  return sms;  // one resident CTA per SM, one query block in flight per CTA
}
