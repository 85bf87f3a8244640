// Peer mappings for the key/value-sharded path: a rank that owns query rows exports its fp32
// accumulator, the other ranks (processes, one per GPU) open it and hand the mapped address to
// sigattn_fwd_shard_acc / sigattn_bwd_shard_acc, whose kernels then add their summands straight
// into the owner's memory (plain reductions and TMA reduce operations; over NVLink when the two
// processes drive different GPUs).  CUDA's inter-process handles name whole allocations, so the
// export also returns the offset of the pointer inside its allocation.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "../../include/sigattn.h"
#include "sigattn_internal.h"

namespace {

typedef CUresult (*GetAddressRangeFn)(CUdeviceptr*, size_t*, CUdeviceptr);

GetAddressRangeFn address_range_fn() {
  static GetAddressRangeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<GetAddressRangeFn>(p);
  }
  return fn;
}

static_assert(sizeof(cudaIpcMemHandle_t) == SIGATTN_PEER_HANDLE_BYTES, "handle size");

}  // namespace

extern "C" {

int sigattn_peer_export(const void* dev_ptr, void* handle, size_t* offset) {
  if (!dev_ptr || !handle || !offset) return SIGATTN_ERR_NULL;
  GetAddressRangeFn range = address_range_fn();
  if (range == nullptr) { sigattn::account(0, SIGATTN_ERR_CUDA, cudaErrorNotSupported); return SIGATTN_ERR_CUDA; }
  CUdeviceptr base = 0;
  size_t size = 0;
  if (range(&base, &size, reinterpret_cast<CUdeviceptr>(dev_ptr)) != CUDA_SUCCESS) {
    sigattn::account(0, SIGATTN_ERR_CUDA, cudaErrorInvalidValue);
    return SIGATTN_ERR_CUDA;
  }
  cudaIpcMemHandle_t h;
  const cudaError_t e = cudaIpcGetMemHandle(&h, reinterpret_cast<void*>(base));
  if (e != cudaSuccess) { sigattn::account(0, SIGATTN_ERR_CUDA, e); return SIGATTN_ERR_CUDA; }
  memcpy(handle, &h, sizeof(h));
  *offset = static_cast<size_t>(reinterpret_cast<CUdeviceptr>(dev_ptr) - base);
  return SIGATTN_OK;
}

int sigattn_peer_open(const void* handle, size_t offset, void** mapped) {
  if (!handle || !mapped) return SIGATTN_ERR_NULL;
  cudaIpcMemHandle_t h;
  memcpy(&h, handle, sizeof(h));
  void* base = nullptr;
  const cudaError_t e = cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess);
  if (e != cudaSuccess) { sigattn::account(0, SIGATTN_ERR_CUDA, e); return SIGATTN_ERR_CUDA; }
  *mapped = static_cast<char*>(base) + offset;
  return SIGATTN_OK;
}

int sigattn_peer_close(void* mapped, size_t offset) {
  if (!mapped) return SIGATTN_ERR_NULL;
  const cudaError_t e = cudaIpcCloseMemHandle(static_cast<char*>(mapped) - offset);
  if (e != cudaSuccess) { sigattn::account(0, SIGATTN_ERR_CUDA, e); return SIGATTN_ERR_CUDA; }
  return SIGATTN_OK;
}

}  // extern "C"
