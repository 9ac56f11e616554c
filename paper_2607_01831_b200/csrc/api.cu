// Status strings, version, device query and workspace status handling.
#include "lynx_common.cuh"

namespace lynx {

int sm_count() {
  static int cached[64] = {0};
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

}  // namespace lynx

extern "C" const char* lynx_status_string(lynx_status s) {
  switch (s) {
    case LYNX_OK: return "ok";
    case LYNX_ERR_NULL: return "a required pointer is NULL";
    case LYNX_ERR_SHAPE: return "invalid or inconsistent size";
    case LYNX_ERR_ALIGN: return "pointer not sufficiently aligned";
    case LYNX_ERR_UNSUPPORTED: return "unsupported shape";
    case LYNX_ERR_WORKSPACE: return "workspace too small";
    case LYNX_ERR_CUDA: return "CUDA runtime error";
    case LYNX_ERR_BAD_BLOCK_TABLE: return "block id out of range seen by a kernel";
    case LYNX_ERR_TIMEOUT: return "a bounded on-chip wait ran out";
    case LYNX_ERR_RANGE: return "a value row has a range beyond what the kernel represents";
  }
  return "unknown status";
}

extern "C" int lynx_version(void) { return 100; }

extern "C" lynx_status lynx_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return LYNX_ERR_NULL;
  if (workspace_bytes < (size_t)lynx::kWsHeaderBytes) return LYNX_ERR_WORKSPACE;
  if (cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return LYNX_ERR_CUDA;
  return LYNX_OK;
}

extern "C" lynx_status lynx_check(void* workspace, void* stream) {
  if (!workspace) return LYNX_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t flags = 0;
  if (cudaMemcpyAsync(&flags, workspace, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LYNX_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LYNX_ERR_CUDA;
  if (flags != 0) {
    if (cudaMemsetAsync(workspace, 0, sizeof(flags), st) != cudaSuccess) return LYNX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LYNX_ERR_CUDA;
  }
  if (flags & lynx::kFlagTimeout) return LYNX_ERR_TIMEOUT;
  if (flags & lynx::kFlagBadBlock) return LYNX_ERR_BAD_BLOCK_TABLE;
  if (flags & lynx::kFlagRange) return LYNX_ERR_RANGE;
  return LYNX_OK;
}
