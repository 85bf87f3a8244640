#include "sigattn_internal.h"
#include "../../include/sigattn.h"
namespace sigattn {
int launch_fwd_bf16(const void*, const void*, const void*, void*, const Problem&, int*, cudaStream_t,
                    unsigned long long*, cudaError_t*) { return SIGATTN_ERR_FLAG; }
}
