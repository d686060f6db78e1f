// Grouped advantage for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc (nor let a framework allocator do it) at
// the point where advantages are needed: a rollout-side process that runs under a frozen memory
// budget next to an inference engine which has claimed the rest of the GPU, a plugin whose host
// application owns every allocation, or code running between the steps of a training loop whose
// allocator must not be disturbed (an allocation can trigger a synchronising free or fragment a
// carefully packed pool).  For them this file carries its own scratch: a fixed array in the
// library's device image, which every GPU that loads the library holds until the process exits.
#include <mutex>
#include "internal.h"

namespace {

constexpr size_t kScratchBytes = 4u << 20;      // 4 MiB, enough for the documented maximum sizes
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};         // device address of g_scratch, per device ordinal
std::mutex g_mutex;

// In host code `g_scratch` only names the symbol; the address a kernel can use has to be asked
// for, once per device, while that device is current.  It is cached for the life of the process
// and would go stale if the application reset the device.
int scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATGRPO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) return ATGRPO_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return ATGRPO_OK;
}

}  // namespace

extern "C" int atgrpo_group_advantages_noalloc(
    const float* rewards, const int32_t* env_id, const int32_t* role_id, const int32_t* turn_id,
    int64_t n_cand, int32_t n_env, int32_t n_role, int32_t n_turn, const atgrpo_params* params,
    float* adv, int32_t* group_of_cand, int32_t* group_offsets, int32_t* group_perm,
    float* group_mean, float* group_std, int32_t* device_status, void* stream) {
  if (!atgrpo::params_ok(params)) return ATGRPO_ERR_INVALID_ARG;
  if (n_cand < 0 || n_env < 1 || n_role < 1 || n_turn < 1) return ATGRPO_ERR_INVALID_ARG;
  const int64_t G = (int64_t)n_env * n_role * n_turn;
  // sizes beyond the fixed scratch are refused before anything is enqueued
  if (n_cand > ATGRPO_NOALLOC_MAX_CAND || G > ATGRPO_NOALLOC_MAX_GROUPS ||
      atgrpo::group_adv_workspace_bytes(n_cand, G) > kScratchBytes)
    return ATGRPO_ERR_UNSUPPORTED;
  if (n_cand > 0 && (rewards == nullptr || env_id == nullptr || role_id == nullptr ||
                     turn_id == nullptr || adv == nullptr))
    return ATGRPO_ERR_INVALID_ARG;
  void* scratch = nullptr;
  const int rc = scratch_address(&scratch);
  if (rc != ATGRPO_OK) return rc;
  // The pipeline zeroes the histogram it needs at the start of every call, so whatever the
  // previous call left in the shared scratch does not matter.
  return atgrpo::group_adv_launch(rewards, env_id, role_id, turn_id, n_cand, n_env, n_role, n_turn,
                                  *params, adv, group_of_cand, group_offsets, group_perm,
                                  group_mean, group_std, device_status, scratch,
                                  static_cast<cudaStream_t>(stream));
}
