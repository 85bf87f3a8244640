// sigattn_bwd_static_scratch: the backward pass for callers that may not allocate device
// memory and so have no workspace to hand to sigattn_bwd.  The fp32 dQ accumulator that
// sigattn_bwd takes from the caller lives here instead, in one fixed file-scope device
// array; everything else (validation, kernels, results) is the ordinary backward.
//
// The array's name is only a host-side handle in host code: its device address is looked
// up once per device with cudaGetSymbolAddress (that device being current) and that
// pointer is what the kernels receive.
#include <mutex>
#include <stdint.h>

#include "../../include/sigattn.h"
#include "sigattn_internal.h"

namespace {

constexpr size_t kMaxElements = size_t(4) << 20;  // 4 Mi fp32 = 16 MiB per device

static __device__ __align__(256) float g_static_dq_accumulator[kMaxElements];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device; resolved on first use per device.
int scratch_for_current_device(float** out, cudaError_t* cuda_err) {
  int dev = 0;
  *cuda_err = cudaGetDevice(&dev);
  if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SIGATTN_ERR_ARCH;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    float* p = nullptr;
    *cuda_err = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_dq_accumulator);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return SIGATTN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

size_t sigattn_bwd_static_scratch_max_elements(void) { return kMaxElements; }

int sigattn_bwd_static_scratch(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk,
                               void* dv, int B, int H, int N, int D, float scale, float bias, int causal,
                               const float* alibi_slopes, int dtype, void* stream) {
  if (!q || !k || !v || !d_o || !dq || !dk || !dv) return SIGATTN_ERR_NULL;
  if (B < 1 || H < 1 || N < 1 || (D != 64 && D != 128)) return SIGATTN_ERR_SHAPE;
  if (static_cast<long long>(B) * H > 65535) return SIGATTN_ERR_SHAPE;
  const unsigned long long elems = static_cast<unsigned long long>(B) * H * static_cast<unsigned long long>(N) * D;
  if (elems > kMaxElements) return SIGATTN_ERR_STATIC_SCRATCH;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return SIGATTN_ERR_ALIGN;
  if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SIGATTN_ERR_ALIGN;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return SIGATTN_ERR_FLAG;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;

  int* status = nullptr;
  if (int rc = sigattn::resolve_device(&status)) return rc;
  cudaError_t ce = cudaSuccess;
  float* scratch = nullptr;
  if (int rc = scratch_for_current_device(&scratch, &ce)) {
    sigattn::account(0, rc, ce);
    return rc;
  }
  sigattn::Problem p{B, H, N, D, scale, bias, causal, alibi_slopes};
  unsigned long long launches = 0;
  int rc;
  if (dtype == SIGATTN_DTYPE_FP32) {
    // the fp32 debug path needs no scratch at all
    rc = sigattn::launch_bwd_fp32(static_cast<const float*>(q), static_cast<const float*>(k),
                                  static_cast<const float*>(v), static_cast<const float*>(d_o),
                                  static_cast<float*>(dq), static_cast<float*>(dk), static_cast<float*>(dv), p,
                                  static_cast<cudaStream_t>(stream), &launches, &ce);
  } else {
    // the launcher clears the elems-long prefix it uses (cudaMemsetAsync on `stream`) before the main kernel
    rc = sigattn::launch_bwd_bf16(q, k, v, d_o, dq, dk, dv, p, scratch, status, static_cast<cudaStream_t>(stream),
                                  &launches, &ce);
  }
  sigattn::account(launches, rc, ce);
  return rc;
}

}  // extern "C"
