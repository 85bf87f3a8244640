// C-ABI layer of libsigattn.so: argument validation, dispatch by dtype, device-side
// status word, error strings.  See include/sigattn.h for the contract.
#include <atomic>
#include <mutex>
#include <stdint.h>

#include "../../include/sigattn.h"
#include "sigattn_internal.h"
#include "sm100_primitives.cuh"

namespace {

__device__ int g_device_status = 0;  // set by kernels when a bounded wait expires

std::atomic<unsigned long long> g_launches{0};
thread_local cudaError_t t_last_cuda = cudaSuccess;

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;                    // guards the two per-device tables below
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
  // Host threads may make their first call on a device together: the tables are filled and read
  // under one lock, so no reader sees the architecture flag without the status pointer.
  std::lock_guard<std::mutex> lock(g_setup_mutex);
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
  if (g_status_ptr[dev] == nullptr) return SIGATTN_ERR_CUDA;   // never launch a kernel that would report to address 0
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

namespace {

// Shared by the scalar-bias and the bias-vector entry points.
// N counts query rows, N_k key/value rows; a causal mask needs N_k >= N (the queries are the last
// N positions, so every query then sees at least one key).
// With pos0_given the caller states where the queries sit relative to key 0 (any value within
// +-2^30; a query before every key then gets zeros), so the N_k >= N rule does not apply.
int check_lengths(int B, int H, int H_kv, int N, int N_k, int D, int causal, int pos0_given, int pos0) {
  if (int rc = check_shape(B, H, N, D)) return rc;
  if (H_kv < 1 || H % H_kv != 0) return SIGATTN_ERR_SHAPE;
  if (int rc = check_shape(B, H_kv, N_k, D)) return rc;
  if (!pos0_given && causal == 1 && N_k < N) return SIGATTN_ERR_SHAPE;
  if (pos0_given && (pos0 > (1 << 30) || pos0 < -(1 << 30))) return SIGATTN_ERR_SHAPE;
  return SIGATTN_OK;
}

int fwd_any(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N, int N_k, int D,
            float scale, float bias, const float* bias_vec, int causal, const float* alibi_slopes, int dtype,
            void* stream, int pos0_given = 0, int pos0 = 0, const int* seqlens = nullptr,
            const float* row_scale = nullptr, float* split_ws = nullptr, int acc_only = 0,
            const int* cu_seqlens = nullptr, int n_seqs = 0) {
  if (!q || !k || !v || (!o && !acc_only)) return SIGATTN_ERR_NULL;
  if (int rc = check_lengths(B, H, H_kv, N, N_k, D, causal, pos0_given, pos0)) return rc;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return SIGATTN_ERR_ALIGN;
  if (alibi_slopes && (reinterpret_cast<uintptr_t>(alibi_slopes) & 3u)) return SIGATTN_ERR_ALIGN;
  if (dtype != SIGATTN_DTYPE_BF16 && dtype != SIGATTN_DTYPE_FP32) return SIGATTN_ERR_FLAG;
  if (acc_only && dtype != SIGATTN_DTYPE_BF16) return SIGATTN_ERR_FLAG;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  sigattn::Problem p{B, H, N, D, scale, bias, causal, alibi_slopes, bias_vec, nullptr, H_kv, N_k, pos0_given, pos0,
                     seqlens, row_scale, split_ws, acc_only, cu_seqlens, n_seqs};
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

int bwd_any(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B, int H,
            int H_kv, int N, int N_k, int D, float scale, float bias, const float* bias_vec, float* dbias, int causal,
            const float* alibi_slopes, int dtype, void* workspace, size_t workspace_bytes, void* stream,
            int pos0_given = 0, int pos0 = 0, const int* seqlens = nullptr, const float* row_scale = nullptr,
            int acc_only = 0, const int* cu_seqlens = nullptr, int n_seqs = 0, float* dtemp = nullptr) {
  if (!q || !k || !v || !d_o || (!dq && !acc_only) || !dk || !dv) return SIGATTN_ERR_NULL;
  if (dtemp && (reinterpret_cast<uintptr_t>(dtemp) & 3u)) return SIGATTN_ERR_ALIGN;
  if (acc_only && dtype != SIGATTN_DTYPE_BF16) return SIGATTN_ERR_FLAG;
  if (int rc = check_lengths(B, H, H_kv, N, N_k, D, causal, pos0_given, pos0)) return rc;
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
  sigattn::Problem p{B, H, N, D, scale, bias, causal, alibi_slopes, bias_vec, dbias, H_kv, N_k, pos0_given, pos0,
                     seqlens, row_scale, nullptr, acc_only, cu_seqlens, n_seqs, dtemp};
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

}  // namespace

extern "C" {

int sigattn_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int D, float scale,
                float bias, int causal, const float* alibi_slopes, int dtype, void* stream) {
  return fwd_any(q, k, v, o, B, H, H, N, N, D, scale, bias, nullptr, causal, alibi_slopes, dtype, stream);
}

int sigattn_fwd_bias_vec(const void* q, const void* k, const void* v, void* o, int B, int H, int N, int D,
                         float scale, const float* bias_bh, int causal, const float* alibi_slopes, int dtype,
                         void* stream) {
  if (!bias_bh) return SIGATTN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(bias_bh) & 3u) return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H, N, N, D, scale, 0.0f, bias_bh, causal, alibi_slopes, dtype, stream);
}

int sigattn_fwd_gqa(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N, int D,
                    float scale, float bias, const float* bias_bh, int causal, const float* alibi_slopes, int dtype,
                    void* stream) {
  if (bias_bh && (reinterpret_cast<uintptr_t>(bias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H_kv, N, N, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream);
}

int sigattn_bwd(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B,
                int H, int N, int D, float scale, float bias, int causal, const float* alibi_slopes, int dtype,
                void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H, N, N, D, scale, bias, nullptr, nullptr, causal, alibi_slopes, dtype,
                 workspace, workspace_bytes, stream);
}

int sigattn_bwd_dtemp(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B,
                      int H, int N, int D, float scale, float bias, const float* bias_bh, int causal,
                      const float* alibi_slopes, int dtype, float* dbias_bh, float* dtemp_bh, void* workspace,
                      size_t workspace_bytes, void* stream) {
  if (!dtemp_bh) return SIGATTN_ERR_NULL;
  if (bias_bh && (reinterpret_cast<uintptr_t>(bias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  if (dbias_bh && (reinterpret_cast<uintptr_t>(dbias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H, N, N, D, scale, bias, bias_bh, dbias_bh, causal, alibi_slopes,
                 dtype, workspace, workspace_bytes, stream, 0, 0, nullptr, nullptr, 0, nullptr, 0, dtemp_bh);
}

int sigattn_bwd_bias_vec(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                         int B, int H, int N, int D, float scale, const float* bias_bh, int causal,
                         const float* alibi_slopes, int dtype, float* dbias_bh, void* workspace,
                         size_t workspace_bytes, void* stream) {
  if (!bias_bh) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H, N, N, D, scale, 0.0f, bias_bh, dbias_bh, causal, alibi_slopes,
                 dtype, workspace, workspace_bytes, stream);
}

int sigattn_bwd_gqa(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B,
                    int H, int H_kv, int N, int D, float scale, float bias, const float* bias_bh, int causal,
                    const float* alibi_slopes, int dtype, float* dbias_bh, void* workspace, size_t workspace_bytes,
                    void* stream) {
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H_kv, N, N, D, scale, bias, bias_bh, dbias_bh, causal, alibi_slopes,
                 dtype, workspace, workspace_bytes, stream);
}

int sigattn_fwd_nk(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N_q, int N_k,
                   int D, float scale, float bias, const float* bias_bh, int causal, const float* alibi_slopes,
                   int dtype, void* stream) {
  if (bias_bh && (reinterpret_cast<uintptr_t>(bias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream);
}

int sigattn_bwd_nk(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv, int B,
                   int H, int H_kv, int N_q, int N_k, int D, float scale, float bias, const float* bias_bh, int causal,
                   const float* alibi_slopes, int dtype, float* dbias_bh, void* workspace, size_t workspace_bytes,
                   void* stream) {
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, dbias_bh, causal,
                 alibi_slopes, dtype, workspace, workspace_bytes, stream);
}

int sigattn_fwd_shard(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N_q, int N_k,
                      int D, float scale, float bias, const float* bias_bh, int causal, int pos0,
                      const float* alibi_slopes, int dtype, void* stream) {
  if (bias_bh && (reinterpret_cast<uintptr_t>(bias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream, 1,
                 pos0);
}

int sigattn_bwd_shard(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                      int B, int H, int H_kv, int N_q, int N_k, int D, float scale, float bias, const float* bias_bh,
                      int causal, int pos0, const float* alibi_slopes, int dtype, float* dbias_bh, void* workspace,
                      size_t workspace_bytes, void* stream) {
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, dbias_bh, causal,
                 alibi_slopes, dtype, workspace, workspace_bytes, stream, 1, pos0);
}

int sigattn_fwd_varlen(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N, int D,
                       float scale, float bias, const float* bias_bh, int causal, const int* seqlens,
                       const float* alibi_slopes, int dtype, void* stream) {
  if (!seqlens) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(seqlens) & 3u) || (reinterpret_cast<uintptr_t>(bias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H_kv, N, N, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream, 0, 0,
                 seqlens);
}

int sigattn_bwd_varlen(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                       int B, int H, int H_kv, int N, int D, float scale, float bias, const float* bias_bh, int causal,
                       const int* seqlens, const float* alibi_slopes, int dtype, float* dbias_bh, void* workspace,
                       size_t workspace_bytes, void* stream) {
  if (!seqlens) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(seqlens) & 3u) || (reinterpret_cast<uintptr_t>(bias_bh) & 3u) ||
      (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H_kv, N, N, D, scale, bias, bias_bh, dbias_bh, causal, alibi_slopes,
                 dtype, workspace, workspace_bytes, stream, 0, 0, seqlens);
}

int sigattn_bwd_set_timing_events(void* start_event, void* stop_event) {
  sigattn::set_bwd_timing_events(static_cast<cudaEvent_t>(start_event), static_cast<cudaEvent_t>(stop_event));
  return SIGATTN_OK;
}

namespace {
size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// sigattn_step_host splits the problem into chunks of whole heads and runs copy-in, kernels
// and copy-out of different chunks on three streams of its own, so that the two directions
// of the host link and the kernels overlap.  Streams and events are created once per device.
constexpr int kHostStepEvents = 64;   // events per kind; head chunking never forms more chunks than this
struct HostStepPipeline {
  cudaStream_t in = nullptr, compute = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done = nullptr;
  cudaEvent_t in_done[kHostStepEvents] = {}, computed[kHostStepEvents] = {};
  bool ready = false;
};
HostStepPipeline g_host_step[kMaxDevices];
std::mutex g_host_step_mutex;

int host_step_pipeline(int dev, HostStepPipeline** out) {
  std::lock_guard<std::mutex> lock(g_host_step_mutex);
  HostStepPipeline& p = g_host_step[dev];
  if (!p.ready) {
    cudaError_t e = cudaSuccess;
    auto stream = [&](cudaStream_t* s) { if (e == cudaSuccess) e = cudaStreamCreateWithFlags(s, cudaStreamNonBlocking); };
    auto event = [&](cudaEvent_t* ev) { if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming); };
    stream(&p.in); stream(&p.compute); stream(&p.out);
    event(&p.start); event(&p.done);
    for (int i = 0; i < kHostStepEvents; ++i) { event(&p.in_done[i]); event(&p.computed[i]); }
    if (e != cudaSuccess) { t_last_cuda = e; return SIGATTN_ERR_CUDA; }
    p.ready = true;
  }
  *out = &p;
  return SIGATTN_OK;
}

// A chunk is either a group of whole batch entries or, within one batch entry, a group of
// heads whose size divides H (so a chunk never straddles two batch entries and the ALiBi slope
// of a head is found at a fixed offset).  About eight chunks are formed, none below 1 MiB per
// tensor unless the whole problem is.
struct HostStepChunking {
  int batches;   // batch entries per chunk (>= 1); heads == H if > 1
  int heads;     // heads per chunk
};
HostStepChunking host_step_chunking(int B, int H, size_t head_bytes) {
  const size_t min_bytes = 1u << 20;
  if (B >= 2 && static_cast<size_t>(H) * head_bytes * B >= 2 * min_bytes && (B >= 8 || H * head_bytes < 8 * min_bytes)) {
    int nb = (B + 7) / 8;
    while (static_cast<size_t>(nb) * H * head_bytes < min_bytes && nb < B) ++nb;
    return {nb, H};
  }
  int best = H;
  for (int d = H; d >= 1; --d) {
    if (H % d != 0) continue;
    if (d * head_bytes < min_bytes && d != H) break;
    if (static_cast<long long>(B) * (H / d) > kHostStepEvents) break;
    best = d;
    if (static_cast<long long>(B) * (H / d) >= 8) break;
  }
  return {1, best};
}
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
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  HostStepPipeline* pipe = nullptr;
  if (int rc = host_step_pipeline(dev, &pipe)) return rc;

  const size_t elem = (dtype == SIGATTN_DTYPE_BF16) ? 2 : 4;
  const size_t head_bytes = static_cast<size_t>(N) * D * elem;   // one (batch, head) slab of a tensor
  const size_t tensor = align256(static_cast<size_t>(B) * H * head_bytes);
  char* base = static_cast<char*>(device_arena);
  float* d_slopes = reinterpret_cast<float*>(base + 8 * tensor);
  char* d_ws = base + 8 * tensor + align256(static_cast<size_t>(H) * sizeof(float));
  const HostStepChunking ck = host_step_chunking(B, H, head_bytes);
  const int chunks_per_batch = H / ck.heads;                       // 1 if chunks are whole batch entries
  const int n_chunks = (ck.batches > 1 || ck.heads == H) ? (B + ck.batches - 1) / ck.batches : B * chunks_per_batch;
  cudaStream_t caller = static_cast<cudaStream_t>(stream);
  const void* in_host[4] = {q_host, k_host, v_host, d_o_host};
  void* out_host[4] = {o_host, dq_host, dk_host, dv_host};
  auto fail = [](cudaError_t e) { t_last_cuda = e; return SIGATTN_ERR_CUDA; };
  cudaError_t e;

  // The three internal streams start after everything already enqueued on the caller's stream.
  if ((e = cudaEventRecord(pipe->start, caller)) != cudaSuccess) return fail(e);
  if ((e = cudaStreamWaitEvent(pipe->in, pipe->start, 0)) != cudaSuccess) return fail(e);
  if ((e = cudaStreamWaitEvent(pipe->compute, pipe->start, 0)) != cudaSuccess) return fail(e);
  if ((e = cudaStreamWaitEvent(pipe->out, pipe->start, 0)) != cudaSuccess) return fail(e);
  if (alibi_slopes_host) {
    e = cudaMemcpyAsync(d_slopes, alibi_slopes_host, static_cast<size_t>(H) * sizeof(float), cudaMemcpyHostToDevice,
                        pipe->in);
    if (e != cudaSuccess) return fail(e);
  }
  for (int c = 0; c < n_chunks; ++c) {
    // chunk c covers `cb` batch entries x `ck.heads` heads starting at (b0, h0)
    const bool whole = (ck.heads == H);
    const int b0 = whole ? c * ck.batches : c / chunks_per_batch;
    const int cb = whole ? (B - b0 < ck.batches ? B - b0 : ck.batches) : 1;
    const int h0 = whole ? 0 : (c % chunks_per_batch) * ck.heads;
    const size_t off = (static_cast<size_t>(b0) * H + h0) * head_bytes;
    const size_t chunk_bytes = static_cast<size_t>(cb) * ck.heads * head_bytes;
    const size_t chunk_ws = sigattn_bwd_workspace_bytes(cb, ck.heads, N, D, dtype);
    const size_t ws_off = (dtype == SIGATTN_DTYPE_BF16) ? off / elem * sizeof(float) : 0;   // fp32 accumulator slab
    for (int i = 0; i < 4; ++i) {
      e = cudaMemcpyAsync(base + i * tensor + off, static_cast<const char*>(in_host[i]) + off, chunk_bytes,
                          cudaMemcpyHostToDevice, pipe->in);
      if (e != cudaSuccess) return fail(e);
    }
    cudaEvent_t in_done = pipe->in_done[c % kHostStepEvents], computed = pipe->computed[c % kHostStepEvents];
    if ((e = cudaEventRecord(in_done, pipe->in)) != cudaSuccess) return fail(e);
    if ((e = cudaStreamWaitEvent(pipe->compute, in_done, 0)) != cudaSuccess) return fail(e);
    const float* slopes = alibi_slopes_host ? d_slopes + h0 : nullptr;
    void* d[8];
    for (int i = 0; i < 8; ++i) d[i] = base + i * tensor + off;
    if (int rc = sigattn_fwd(d[0], d[1], d[2], d[4], cb, ck.heads, N, D, scale, bias, causal, slopes, dtype,
                             pipe->compute))
      return rc;
    if (int rc = sigattn_bwd(d[0], d[1], d[2], d[3], d[5], d[6], d[7], cb, ck.heads, N, D, scale, bias, causal, slopes,
                             dtype, chunk_ws ? d_ws + ws_off : nullptr, chunk_ws, pipe->compute))
      return rc;
    if ((e = cudaEventRecord(computed, pipe->compute)) != cudaSuccess) return fail(e);
    if ((e = cudaStreamWaitEvent(pipe->out, computed, 0)) != cudaSuccess) return fail(e);
    for (int i = 0; i < 4; ++i) {
      e = cudaMemcpyAsync(static_cast<char*>(out_host[i]) + off, base + (4 + i) * tensor + off, chunk_bytes,
                          cudaMemcpyDeviceToHost, pipe->out);
      if (e != cudaSuccess) return fail(e);
    }
  }
  // The last copies out follow the last kernels, which follow the last copies in.
  if ((e = cudaEventRecord(pipe->done, pipe->out)) != cudaSuccess) return fail(e);
  if ((e = cudaStreamWaitEvent(caller, pipe->done, 0)) != cudaSuccess) return fail(e);
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

int sigattn_fwd_rowscale(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N_q,
                         int N_k, int D, float scale, float bias, const float* bias_bh, int causal,
                         const float* row_scale, const float* alibi_slopes, int dtype, void* stream) {
  if (!row_scale) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(row_scale) & 3u) || (reinterpret_cast<uintptr_t>(bias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream, 0, 0,
                 nullptr, row_scale);
}

int sigattn_bwd_rowscale(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                         int B, int H, int H_kv, int N_q, int N_k, int D, float scale, float bias,
                         const float* bias_bh, int causal, const float* row_scale, const float* alibi_slopes,
                         int dtype, float* dbias_bh, void* workspace, size_t workspace_bytes, void* stream) {
  if (!row_scale) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(row_scale) & 3u) || (reinterpret_cast<uintptr_t>(bias_bh) & 3u) ||
      (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, dbias_bh, causal,
                 alibi_slopes, dtype, workspace, workspace_bytes, stream, 0, 0, nullptr, row_scale);
}

int sigattn_fwd_shard_acc(const void* q, const void* k, const void* v, float* o_acc, int B, int H, int H_kv, int N_q,
                          int N_k, int D, float scale, float bias, const float* bias_bh, int causal, int pos0,
                          const float* alibi_slopes, int dtype, void* stream) {
  if (!o_acc) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(o_acc) & 15u) || (reinterpret_cast<uintptr_t>(bias_bh) & 3u)) return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, nullptr, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream,
                 1, pos0, nullptr, nullptr, o_acc, 1);
}

int sigattn_bwd_shard_acc(const void* q, const void* k, const void* v, const void* d_o, float* dq_acc, void* dk,
                          void* dv, int B, int H, int H_kv, int N_q, int N_k, int D, float scale, float bias,
                          const float* bias_bh, int causal, int pos0, const float* alibi_slopes, int dtype,
                          float* dbias_bh, void* stream) {
  if (!dq_acc) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, nullptr, dk, dv, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, dbias_bh, causal,
                 alibi_slopes, dtype, dq_acc, sigattn_bwd_workspace_bytes(B, H, N_q, D, dtype), stream, 1, pos0, nullptr,
                 nullptr, 1);
}

int sigattn_bwd_shard_acc_kv(const void* q, const void* k, const void* v, const void* d_o, float* dq_acc, void* dk,
                             void* dv, int B, int H, int H_kv, int N_q, int N_k, int D, float scale, float bias,
                             const float* bias_bh, int causal, int pos0, const float* alibi_slopes, int dtype,
                             float* dbias_bh, void* stream) {
  if (!dq_acc) return SIGATTN_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(bias_bh) & 3u) || (reinterpret_cast<uintptr_t>(dbias_bh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, nullptr, dk, dv, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, dbias_bh, causal,
                 alibi_slopes, dtype, dq_acc, sigattn_bwd_workspace_bytes(B, H, N_q, D, dtype), stream, 1, pos0, nullptr,
                 nullptr, 2);
}

int sigattn_check_cu_seqlens(const int* host_cu_seqlens, int n_seqs, int T) {
  if (!host_cu_seqlens) return SIGATTN_ERR_NULL;
  if (n_seqs < 1 || T < 1) return SIGATTN_ERR_SHAPE;
  if (host_cu_seqlens[0] != 0 || host_cu_seqlens[n_seqs] != T) return SIGATTN_ERR_SHAPE;
  for (int s = 0; s < n_seqs; ++s)
    if (host_cu_seqlens[s + 1] < host_cu_seqlens[s]) return SIGATTN_ERR_SHAPE;
  return SIGATTN_OK;
}

int sigattn_acc_to_bf16(const float* acc, void* out, size_t n, float mul, void* stream) {
  if (!acc || !out) return SIGATTN_ERR_NULL;
  if (!aligned16(acc) || !aligned16(out)) return SIGATTN_ERR_ALIGN;
  if (n == 0 || n % 4 != 0) return SIGATTN_ERR_SHAPE;
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  unsigned long long launches = 0;
  cudaError_t ce = cudaSuccess;
  const int rc = sigattn::launch_acc_to_bf16(acc, out, n, mul, static_cast<cudaStream_t>(stream), &launches, &ce);
  g_launches.fetch_add(launches);
  if (rc == SIGATTN_ERR_CUDA) t_last_cuda = ce;
  return rc;
}

int sigattn_fwd_ragged(const void* q, const void* k, const void* v, void* o, int H, int H_kv, int T, int D,
                       const int* cu_seqlens, int n_seqs, float scale, float bias, const float* bias_sh, int causal,
                       const float* alibi_slopes, int dtype, void* stream) {
  if (!cu_seqlens) return SIGATTN_ERR_NULL;
  if (n_seqs < 1) return SIGATTN_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(cu_seqlens) & 3u) || (reinterpret_cast<uintptr_t>(bias_sh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return fwd_any(q, k, v, o, 1, H, H_kv, T, T, D, scale, bias, bias_sh, causal, alibi_slopes, dtype, stream, 0, 0,
                 nullptr, nullptr, nullptr, 0, cu_seqlens, n_seqs);
}

int sigattn_bwd_ragged(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                       int H, int H_kv, int T, int D, const int* cu_seqlens, int n_seqs, float scale, float bias,
                       const float* bias_sh, int causal, const float* alibi_slopes, int dtype, float* dbias_sh,
                       void* workspace, size_t workspace_bytes, void* stream) {
  if (!cu_seqlens) return SIGATTN_ERR_NULL;
  if (n_seqs < 1) return SIGATTN_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(cu_seqlens) & 3u) || (reinterpret_cast<uintptr_t>(bias_sh) & 3u) ||
      (reinterpret_cast<uintptr_t>(dbias_sh) & 3u))
    return SIGATTN_ERR_ALIGN;
  return bwd_any(q, k, v, d_o, dq, dk, dv, 1, H, H_kv, T, T, D, scale, bias, bias_sh, dbias_sh, causal, alibi_slopes,
                 dtype, workspace, workspace_bytes, stream, 0, 0, nullptr, nullptr, 0, cu_seqlens, n_seqs);
}

size_t sigattn_fwd_decode_workspace_bytes(int B, int H, int N_q, int D, int dtype) {
  if (check_shape(B, H, N_q, D) != SIGATTN_OK) return 0;
  if (dtype != SIGATTN_DTYPE_BF16) return 0;
  return static_cast<size_t>(B) * H * N_q * D * sizeof(float);
}

int sigattn_fwd_decode(const void* q, const void* k, const void* v, void* o, int B, int H, int H_kv, int N_q, int N_k,
                       int D, float scale, float bias, const float* bias_bh, int causal, const float* alibi_slopes,
                       int dtype, void* workspace, size_t workspace_bytes, void* stream) {
  if (reinterpret_cast<uintptr_t>(bias_bh) & 3u) return SIGATTN_ERR_ALIGN;
  const size_t need = sigattn_fwd_decode_workspace_bytes(B, H, N_q, D, dtype);
  if (need > 0) {
    if (!workspace) return SIGATTN_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SIGATTN_ERR_ALIGN;
    if (workspace_bytes < need) return SIGATTN_ERR_WORKSPACE;
  }
  return fwd_any(q, k, v, o, B, H, H_kv, N_q, N_k, D, scale, bias, bias_bh, causal, alibi_slopes, dtype, stream, 0, 0,
                 nullptr, nullptr, need > 0 ? static_cast<float*>(workspace) : nullptr);
}

int sigattn_seqlen_norm(float* row_scale, int N_q, int N_k, float alpha, int causal, void* stream) {
  if (!row_scale) return SIGATTN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(row_scale) & 3u) return SIGATTN_ERR_ALIGN;
  if (N_q < 1 || N_k < 1 || (causal == 1 && N_k < N_q)) return SIGATTN_ERR_SHAPE;
  if (causal != 0 && causal != 1) return SIGATTN_ERR_FLAG;
  int dev = 0;
  int* status = nullptr;
  if (int rc = device_setup(&dev, &status)) return rc;
  unsigned long long launches = 0;
  cudaError_t ce = cudaSuccess;
  const int rc = sigattn::launch_seqlen_norm(row_scale, N_q, N_k, N_k - N_q, causal, alpha,
                                             static_cast<cudaStream_t>(stream), &launches, &ce);
  g_launches.fetch_add(launches);
  if (rc == SIGATTN_ERR_CUDA) t_last_cuda = ce;
  return rc;
}

}  // extern "C"
