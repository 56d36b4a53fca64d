// Error bookkeeping, device queries and small host-only entry points.
#include "common.cuh"

#include <mutex>

namespace specvlm {

static thread_local std::string g_last_error = "";

int fail(int code, const std::string& msg) {
  g_last_error = msg;
  return code;
}

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return SPECVLM_OK;
  return fail(SPECVLM_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

int sm_count() {
  static int cached[64];
  static std::once_flag once;
  std::call_once(once, [] { for (int& c : cached) c = 0; });
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace specvlm

extern "C" int specvlm_version(void) { return SPECVLM_VERSION; }

extern "C" const char* specvlm_last_error_string(void) { return specvlm::g_last_error.c_str(); }

extern "C" int specvlm_workspace_init(void* workspace, size_t bytes, void* stream) {
  SPECVLM_REQUIRE(workspace != nullptr || bytes == 0, "workspace_init: null workspace");
  if (bytes == 0) return SPECVLM_OK;
  return specvlm::check_cuda(cudaMemsetAsync(workspace, 0, bytes, static_cast<cudaStream_t>(stream)),
                             "workspace_init memset");
}

extern "C" int specvlm_tree_validate_host(const int32_t* parent, const int32_t* tokens, int T) {
  if (parent == nullptr || T < 1 || T > SPECVLM_MAX_TREE)
    return specvlm::fail(SPECVLM_ERR_BAD_TREE, "tree_validate: need 1 <= T <= 64 and a parent array");
  if (parent[0] != -1) return specvlm::fail(SPECVLM_ERR_BAD_TREE, "tree_validate: parent[0] must be -1");
  for (int i = 1; i < T; ++i)
    if (parent[i] < 0 || parent[i] >= i)
      return specvlm::fail(SPECVLM_ERR_BAD_TREE, "tree_validate: parent[i] must lie in [0, i)");
  if (tokens != nullptr)
    for (int i = 1; i < T; ++i)
      for (int j = i + 1; j < T; ++j)
        if (parent[i] == parent[j] && tokens[i] == tokens[j])
          return specvlm::fail(SPECVLM_ERR_BAD_TREE, "tree_validate: siblings share a token");
  return SPECVLM_OK;
}
