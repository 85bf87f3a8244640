// C-ABI layer of libsigattn.so: argument validation, dispatch by dtype, device-side
// status word, error strings.  See include/sigattn.h for the contract.
#include <atomic>
#include <stdint.h>

#include "../../include/sigattn.h"
#include "sigattn_internal.h"
#include "sm100_primitives.cuh"

namespace {

__device__ int g_device_status = 0;  // set by kernels when a bounded wait expires

std::atomic<unsigned long long> g_launches{0};
thread_local cudaError_t t_last_cuda = cudaSuccess;

constexpr int kMaxDevices = 64;
int* g_status_ptr[kMaxDevices] = {nullptr};
int g_arch_ok[kMaxDevices] = {0};  // 0 unknown, 1 sm_100, -1 other

// One warp waits on a barrier that is never signalled; the bounded wait must expire, the
// kernel must return, and the status word must say so.
__global__ void selftest_bounded_wait_kernel(long long limit_cycles, int* status) {
  __shared__ uint64_t bar;
  __shared__ int cta_err;
  if (threadIdx.x == 0) {
    cta_err = 0;
    sm100::mbar_init(sm100::smem_u32(&bar), 1);
    sm100::fence_mbar_init();
  }
  __syncthreads();
  const bool ok = sm100::mbar_wait_limit(sm100::smem_u32(&bar), 0, &cta_err, 1, limit_cycles);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || cta_err != 0)) atomicExch(status, 900 + cta_err);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Resolve per-device facts once: compute capability and the address of the status word.
int device_setup(int* dev_out, int** status_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return SIGATTN_ERR_ARCH;
  if (g_arch_ok[dev] == 0) {
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
    int* sp = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&sp), g_device_status);
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
    g_status_ptr[dev] = sp;
    g_arch_ok[dev] = (major == 10) ? 1 : -1;
  }
  if (g_arch_ok[dev] != 1) return SIGATTN_ERR_ARCH;
  *dev_out = dev;
  *status_out = g_status_ptr[dev];
  return SIGATTN_OK;
}

int check_shape(int B, int H, int N, int D) {
  if (B < 1 || H < 1 || N < 1) return SIGATTN_ERR_SHAPE;
  if (D != 64 && D != 128) return SIGATTN_ERR_SHAPE;
  const long long bh = static_cast<long long>(B) * H;
  if (bh > 65535) return SIGATTN_ERR_SHAPE;                           // grid.y and TMA extent budget
  if (bh * static_cast<long long>(N) >= (1ll << 31)) return SIGATTN_ERR_SHAPE;  // row index must fit int32
  return SIGATTN_OK;
}

}  // namespace

namespace sigattn {

int resolve_device(int** status) {
  int dev = 0;
  return device_setup(&dev, status);
}

void account(unsigned long long launches, int rc, cudaError_t cuda_err) {
  g_launches.fetch_add(launches);
  if (rc == SIGATTN_ERR_CUDA) t_last_cuda = cuda_err;
}

}  // namespace sigattn

extern "C" {

int sigattn_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int D, float scale,
                float bias, int causal, const float* alibi_slopes, int dtype, void* stream) {
  if (!q || !k || !v || !o) return SIGATTN_ERR_NULL;
  if (int rc = check_shape(B, H, N, D)) return rc;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return SIGATTN_ERR_ALIGN;
  if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SIGATTN_ERR_ALIGN;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return SIGATTN_ERR_FLAG;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  sigattn::Problem p{B, H, N, D, scale, bias, causal, alibi_slopes};
  unsigned long long launches = 0;
  cudaError_t ce = cudaSuccess;
  int rc;
  if (dtype == SIGATTN_DTYPE_FP32) {
    rc = sigattn::launch_fwd_fp32(static_cast<const float*>(q), static_cast<const float*>(k),
                                  static_cast<const float*>(v), static_cast<float*>(o), p,
                                  static_cast<cudaStream_t>(stream), &launches, &ce);
  } else {
    rc = sigattn::launch_fwd_bf16(q, k, v, o, p, status, static_cast<cudaStream_t>(stream), &launches, &ce);
  }
  g_launches.fetch_add(launches);
  if (rc == SIGATTN_ERR_CUDA) t_last_cuda = ce;
  return rc;
}

int sigattn_bwd(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B,
                int H, int N, int D, float scale, float bias, int causal, const float* alibi_slopes, int dtype,
                void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !k || !v || !d_o || !dq || !dk || !dv) return SIGATTN_ERR_NULL;
  if (int rc = check_shape(B, H, N, D)) return rc;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return SIGATTN_ERR_ALIGN;
  if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SIGATTN_ERR_ALIGN;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return SIGATTN_ERR_FLAG;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;
  const size_t need = sigattn_bwd_workspace_bytes(B, H, N, D, dtype);
  if (need > 0) {
    if (!workspace) return SIGATTN_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SIGATTN_ERR_ALIGN;
    if (workspace_bytes < need) return SIGATTN_ERR_WORKSPACE;
  }
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  sigattn::Problem p{B, H, N, D, scale, bias, causal, alibi_slopes};
  unsigned long long launches = 0;
  cudaError_t ce = cudaSuccess;
  int rc;
  if (dtype == SIGATTN_DTYPE_FP32) {
    rc = sigattn::launch_bwd_fp32(static_cast<const float*>(q), static_cast<const float*>(k),
                                  static_cast<const float*>(v), static_cast<const float*>(d_o),
                                  static_cast<float*>(dq), static_cast<float*>(dk), static_cast<float*>(dv), p,
                                  static_cast<cudaStream_t>(stream), &launches, &ce);
  } else {
    rc = sigattn::launch_bwd_bf16(q, k, v, d_o, dq, dk, dv, p, workspace, status,
                                  static_cast<cudaStream_t>(stream), &launches, &ce);
  }
  g_launches.fetch_add(launches);
  if (rc == SIGATTN_ERR_CUDA) t_last_cuda = ce;
  return rc;
}

int sigattn_bwd_set_timing_events(void* start_event, void* stop_event) {
  sigattn::set_bwd_timing_events(static_cast<cudaEvent_t>(start_event), static_cast<cudaEvent_t>(stop_event));
  return SIGATTN_OK;
}

namespace {
size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
}

size_t sigattn_step_host_arena_bytes(int B, int H, int N, int D, int dtype) {
  if (check_shape(B, H, N, D) != SIGATTN_OK) return 0;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return 0;
  const size_t tensor = align256(static_cast<size_t>(B) * H * N * D * (dtype == SIGATTN_DTYPE_BF16 ? 2 : 4));
  return 8 * tensor + align256(static_cast<size_t>(H) * sizeof(float)) +
         align256(sigattn_bwd_workspace_bytes(B, H, N, D, dtype));
}

int sigattn_step_host(const void* q_host, const void* k_host, const void* v_host, const void* d_o_host, void* o_host,
                      void* dq_host, void* dk_host, void* dv_host, int B, int H, int N, int D, float scale,
                      float bias, int causal, const float* alibi_slopes_host, int dtype, void* device_arena,
                      size_t arena_bytes, void* stream) {
  if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !dq_host || !dk_host || !dv_host || !device_arena)
    return SIGATTN_ERR_NULL;
  if (int rc = check_shape(B, H, N, D)) return rc;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return SIGATTN_ERR_FLAG;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;
  if (reinterpret_cast<uintptr_t>(device_arena) & 255u) return SIGATTN_ERR_ALIGN;
  if (arena_bytes < sigattn_step_host_arena_bytes(B, H, N, D, dtype)) return SIGATTN_ERR_WORKSPACE;
  const size_t bytes = static_cast<size_t>(B) * H * N * D * (dtype == SIGATTN_DTYPE_BF16 ? 2 : 4);
  const size_t tensor = align256(bytes);
  char* base = static_cast<char*>(device_arena);
  void* d[8];
  for (int i = 0; i < 8; ++i) d[i] = base + i * tensor;
  float* d_slopes = reinterpret_cast<float*>(base + 8 * tensor);
  void* d_ws = base + 8 * tensor + align256(static_cast<size_t>(H) * sizeof(float));
  const size_t ws_bytes = sigattn_bwd_workspace_bytes(B, H, N, D, dtype);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const void* in_host[4] = {q_host, k_host, v_host, d_o_host};
  for (int i = 0; i < 4; ++i) {
    cudaError_t e = cudaMemcpyAsync(d[i], in_host[i], bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  }
  if (alibi_slopes_host) {
    cudaError_t e = cudaMemcpyAsync(d_slopes, alibi_slopes_host, static_cast<size_t>(H) * sizeof(float),
                                    cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  }
  const float* slopes = alibi_slopes_host ? d_slopes : nullptr;
  if (int rc = sigattn_fwd(d[0], d[1], d[2], d[4], B, H, N, D, scale, bias, causal, slopes, dtype, stream)) return rc;
  if (int rc = sigattn_bwd(d[0], d[1], d[2], d[3], d[5], d[6], d[7], B, H, N, D, scale, bias, causal, slopes, dtype,
                           ws_bytes ? d_ws : nullptr, ws_bytes, stream))
    return rc;
  void* out_host[4] = {o_host, dq_host, dk_host, dv_host};
  for (int i = 0; i < 4; ++i) {
    cudaError_t e = cudaMemcpyAsync(out_host[i], d[4 + i], bytes, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  }
  return SIGATTN_OK;
}

size_t sigattn_bwd_workspace_bytes(int B, int H, int N, int D, int dtype) {
  if (check_shape(B, H, N, D) != SIGATTN_OK) return 0;
  if (dtype != SIGATTN_DTYPE_BF16) return 0;
  return sigattn::bwd_bf16_workspace_bytes(B, H, N, D);
}

int sigattn_check(void* stream) {
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  int host_status = 0;
  e = cudaMemcpy(&host_status, status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  if (host_status != 0) {
    e = cudaMemset(status, 0, sizeof(int));
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
    return SIGATTN_ERR_DEVICE_TIMEOUT;
  }
  return SIGATTN_OK;
}

int sigattn_selftest_bounded_wait(int limit_us, void* stream) {
  if (limit_us < 1 || limit_us > 100000) return SIGATTN_ERR_FLAG;
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  int khz = 0;
  cudaError_t e = cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev);
  if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  const long long limit_cycles = static_cast<long long>(limit_us) * khz / 1000;
  selftest_bounded_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles, status);
  e = cudaGetLastError();
  if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
  g_launches.fetch_add(1);
  return SIGATTN_OK;
}

const char* sigattn_strerror(int code) {
  switch (code) {
    case SIGATTN_OK: return "success";
    case SIGATTN_ERR_NULL: return "null pointer argument";
    case SIGATTN_ERR_SHAPE: return "unsupported shape (D must be 64 or 128; B, H, N >= 1; B*H <= 65535; B*H*N < 2^31)";
    case SIGATTN_ERR_ALIGN: return "misaligned pointer (tensors 16 bytes, workspace 256 bytes, slopes 4 bytes)";
    case SIGATTN_ERR_FLAG: return "bad dtype or flag";
    case SIGATTN_ERR_WORKSPACE: return "workspace too small (see sigattn_bwd_workspace_bytes)";
    case SIGATTN_ERR_ARCH: return "device is not sm_100 (B200)";
    case SIGATTN_ERR_CUDA: return "CUDA runtime or driver error (see sigattn_last_cuda_error)";
    case SIGATTN_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired; results of that launch are invalid";
    case SIGATTN_ERR_STATIC_SCRATCH: return "problem larger than the built-in scratch of sigattn_bwd_static_scratch (B*H*N*D elements over the limit)";
    default: return "unknown sigattn error code";
  }
}

const char* sigattn_last_cuda_error(void) { return cudaGetErrorString(t_last_cuda); }

int sigattn_version(void) { return 100; }

unsigned long long sigattn_launch_count(void) { return g_launches.load(); }

}  // extern "C"
