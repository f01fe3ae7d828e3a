// Library identification and status strings.
#include "../../include/specvlm.h"

extern "C" const char* specvlm_version(void) { return "specvlm-b200 0.1 (sm_100a)"; }

extern "C" const char* specvlm_status_string(int32_t status) {
  switch (status) {
    case SPECVLM_OK: return "ok";
    case SPECVLM_ERR_INVALID_ARG: return "invalid argument";
    case SPECVLM_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case SPECVLM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SPECVLM_ERR_CUDA: return "CUDA call failed";
    case SPECVLM_ERR_TIMEOUT: return "device-side wait timed out";
    case SPECVLM_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of a no-allocation call";
    default: return "unknown status";
  }
}
