// placeholder until the tcgen05 kernels land
#include "citrus_internal.h"
namespace citrus {
cudaError_t tc_init() { return cudaErrorNotSupported; }
cudaError_t tc_attention(const QueryRows&, const Candidates&, void*, float*, int, int*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t tc_score_lse(const QueryRows&, const Candidates&, float*, float*, float*, int, int*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t tc_colsum(const QueryRows&, const Candidates&, const float*, int, float*, int, int*, cudaStream_t) { return cudaErrorNotSupported; }
}
