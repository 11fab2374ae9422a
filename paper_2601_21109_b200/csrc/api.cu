// Status strings and version of the C ABI.
#include "cwl_common.cuh"

extern "C" const char* cwl_status_string(cwl_status s) {
  switch (s) {
    case CWL_OK: return "ok";
    case CWL_ERR_INVALID_ARG: return "invalid argument";
    case CWL_ERR_SHAPE: return "bad leading dimension or alignment";
    case CWL_ERR_UNSUPPORTED: return "unsupported shape";
    case CWL_ERR_CAPACITY: return "chunk table capacity exceeded";
    case CWL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CWL_ERR_CUDA: return "CUDA call failed";
    case CWL_ERR_TIMEOUT: return "bounded device-side wait ran out";
  }
  return "unknown status";
}

extern "C" int cwl_version(void) { return 100; }
