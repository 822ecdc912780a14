#include "jet_common.cuh"

extern "C" const char* jet_status_string(jet_status s) {
  switch (s) {
    case JET_OK: return "JET_OK";
    case JET_ERR_INVALID_ARG: return "JET_ERR_INVALID_ARG";
    case JET_ERR_UNSUPPORTED: return "JET_ERR_UNSUPPORTED";
    case JET_ERR_WORKSPACE: return "JET_ERR_WORKSPACE";
    case JET_ERR_CUDA: return "JET_ERR_CUDA";
    case JET_ERR_TIMEOUT: return "JET_ERR_TIMEOUT";
    default: return "JET_ERR_UNKNOWN";
  }
}
