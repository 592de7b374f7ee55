#include "attn_common.cuh"
using namespace sepllm;
extern "C" sepllm_status sepllm_attn_bwd(const sepllm_attn_desc* desc, const sepllm_index_desc* idesc,
                              const void* dO, const void* Q, const void* K, const void* V,
                              const void* O, const float* LSE, const void* index, void* dQ,
                              void* dK, void* dV, void* workspace, void* stream) {
  return SEPLLM_NOT_BUILT;
}
