#include "sigattn_internal.h"
#include "../../include/sigattn.h"
namespace sigattn {
int launch_bwd_bf16(const void*, const void*, const void*, const void*, void*, void*, void*, const Problem&, void*,
                    int*, cudaStream_t, unsigned long long*, cudaError_t*) { return SIGATTN_ERR_FLAG; }
size_t bwd_bf16_workspace_bytes(int B, int H, int N, int D) { return (size_t)B * H * N * D * 4; }
}
