// Entry points that do not belong to one kernel family.
#include "attn_common.cuh"

using namespace sepllm;

extern "C" const char* sepllm_status_string(sepllm_status s) {
  switch (s) {
    case SEPLLM_OK: return "ok";
    case SEPLLM_INVALID_ARG: return "invalid argument";
    case SEPLLM_UNSUPPORTED: return "unsupported configuration";
    case SEPLLM_BUFFER_TOO_SMALL: return "buffer too small";
    case SEPLLM_CUDA_ERROR: return "CUDA error";
    case SEPLLM_CAPACITY_EXCEEDED: return "side capacity exceeded";
    case SEPLLM_TIMEOUT: return "device wait timed out";
    case SEPLLM_NOT_BUILT: return "not built";
    default: return "unknown status";
  }
}

extern "C" sepllm_status sepllm_last_device_status(const void* buffer, int32_t* out,
                                                   void* stream_) {
  if (!buffer || !out) return SEPLLM_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  SEPLLM_CUDA_TRY(cudaMemcpyAsync(out, buffer, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  SEPLLM_CUDA_TRY(cudaStreamSynchronize(stream));
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_attn_workspace_bytes(const sepllm_attn_desc* desc,
                                                     const sepllm_index_desc* idesc,
                                                     size_t* fwd_bytes, size_t* bwd_bytes) {
  sepllm_status st = check_attn(desc, idesc);
  if (st != SEPLLM_OK) return st;
  const AttnLayout lay = attn_layout(desc, idesc);
  if (fwd_bytes) *fwd_bytes = lay.fwd_bytes;
  if (bwd_bytes) *bwd_bytes = lay.bwd_bytes;
  return SEPLLM_OK;
}
