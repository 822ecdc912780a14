#include "jet_common.cuh"
extern "C" size_t jet_tree_verify_attn_workspace_bytes(int, int, int, int, int, int) { return 256; }
extern "C" jet_status jet_tree_verify_attn(const void*, const void*, const void*, const int32_t*, int, int,
                                           int64_t, const int32_t*, int, const void*, const void*,
                                           const uint32_t*, const int32_t*, int, int, int, int, int,
                                           int64_t, float, void*, float*, int32_t*, void*, size_t, void*) {
  return JET_ERR_UNSUPPORTED;
}
