// tcgen05 Gram path (placeholder until the tensor-core kernel lands).
#include "common.cuh"

bool cdg_umma_supported(int, long long, int) { return false; }
int cdg_umma_setup(cdgrab_ctx *) { return CDGRAB_ERR_INVALID; }
void cdg_umma_teardown(cdgrab_ctx *) {}
cudaError_t cdg_launch_gram_umma(cdgrab_ctx *, const void *, cudaStream_t) { return cudaErrorNotSupported; }
