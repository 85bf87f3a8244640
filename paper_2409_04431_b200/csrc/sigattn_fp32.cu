// float32 debug path on CUDA cores: the definition evaluated with exact expf and a
// true division, fp32 FMA accumulation, no tensor cores (TF32 would cost 1e-3 of
// accuracy).  One thread block per query row (forward, dQ) or per key row (dK, dV);
// nothing is shared between blocks, so every tensor output is deterministic (the optional
// bias gradient is a sum over all blocks of a head and is added with fp32 atomics).
//
// N counts query rows, N_k key/value rows; query i has position i + off relative to key 0
// (off = N_k - N when the queries are the last N positions, 0 for self-attention; any value,
// also negative, for a shard of keys and values).
//
// Forward: Eq. 3 / Algorithm 1.  Backward: the sigmoid column of the forward/backward
// table in Appendix F.1 / Algorithm 2, with the factor scale = 1/sqrt(d) in dQ and dK.
#include "sigattn_internal.h"
#include "../../include/sigattn.h"

namespace sigattn {
namespace {

constexpr int kThreads = 128;

__device__ __forceinline__ float sigmoid_exact(float x) { return 1.0f / (1.0f + expf(-x)); }

// P (1 - P) evaluated as sigmoid(x) * sigmoid(-x): the same quantity (1 - sigmoid(x) =
// sigmoid(-x)), but without the cancellation of 1 - P when P rounds to 1.
__device__ __forceinline__ float sigmoid_slope(float x) { return sigmoid_exact(x) * sigmoid_exact(-x); }

__device__ __forceinline__ float dot_row(const float* __restrict__ a_smem, const float* __restrict__ b, int D) {
  float s = 0.0f;
  for (int d = 0; d < D; ++d) s = fmaf(a_smem[d], b[d], s);
  return s;
}

// Batch stored without padding: the sequence that owns `row` (largest s with cu[s] <= row).
__device__ __forceinline__ int seq_of_row_fp32(const int* __restrict__ cu, int n_seqs, int row) {
  int lo = 0, hi = n_seqs;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= row) lo = mid; else hi = mid;
  }
  return lo;
}

// grid (N, B*H); block 128.  Thread t handles key j0 + t, then output column t.
__global__ void fwd_fp32_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                const float* __restrict__ v, float* __restrict__ o, int H, int N, int D,
                                float scale, float bias, int causal, const float* __restrict__ slopes,
                                const float* __restrict__ bias_vec, int H_kv, int N_k, int off,
                                const int* __restrict__ seqlens, const float* __restrict__ row_scale,
                                const int* __restrict__ cu, int n_seqs) {
  __shared__ float sq[128];
  __shared__ float sp[kThreads];
  const int i = blockIdx.x, bh = blockIdx.y, t = threadIdx.x;
  const int sq_id = cu ? seq_of_row_fp32(cu, n_seqs, i) : 0;
  if (bias_vec) bias = bias_vec[cu ? sq_id * H + bh : bh];
  const size_t base = static_cast<size_t>(bh) * N * D;
  const size_t kv_base = static_cast<size_t>((bh / H) * H_kv + (bh % H) / (H / H_kv)) * N_k * D;
  const float slope = slopes ? slopes[bh % H] : 0.0f;
  if (t < D) sq[t] = q[base + static_cast<size_t>(i) * D + t];
  __syncthreads();
  // padded batch: keys past the sequence's length carry no weight, rows past it are zero
  const int n_valid = seqlens ? max(0, min(N, seqlens[bh / H])) : N_k;
  int jend = (i >= n_valid && seqlens) ? 0 : min(n_valid, causal ? max(0, min(N_k, i + off + 1)) : N_k);
  const int jbeg = cu ? cu[sq_id] : 0;          // batch without padding: keys of the row's own sequence only
  if (cu) jend = min(jend, cu[sq_id + 1]);
  float acc = 0.0f;
  for (int j0 = jbeg; j0 < jend; j0 += kThreads) {
    const int j = j0 + t;
    float p = 0.0f;
    if (j < jend) {
      const float s = dot_row(sq, k + kv_base + static_cast<size_t>(j) * D, D);
      const float x = fmaf(scale, s, bias) - slope * fabsf(static_cast<float>(i + off - j));
      p = sigmoid_exact(x);
    }
    sp[t] = p;
    __syncthreads();
    if (t < D) {
      const int cnt = min(kThreads, jend - j0);
      for (int jj = 0; jj < cnt; ++jj) acc = fmaf(sp[jj], v[kv_base + static_cast<size_t>(j0 + jj) * D + t], acc);
    }
    __syncthreads();
  }
  if (t < D) o[base + static_cast<size_t>(i) * D + t] = row_scale ? row_scale[i] * acc : acc;
}

// dQ_i = scale * sum_j dS_ij K_j.  grid (N, B*H).
__global__ void bwd_dq_fp32_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                   const float* __restrict__ v, const float* __restrict__ d_o,
                                   float* __restrict__ dq, int H, int N, int D, float scale, float bias,
                                   int causal, const float* __restrict__ slopes,
                                   const float* __restrict__ bias_vec, float* __restrict__ dbias, int H_kv,
                                   int N_k, int off, const int* __restrict__ seqlens,
                                   const float* __restrict__ row_scale, const int* __restrict__ cu, int n_seqs) {
  __shared__ float sq[128];
  __shared__ float sdo[128];
  __shared__ float sds[kThreads];
  const int i = blockIdx.x, bh = blockIdx.y, t = threadIdx.x;
  const int sq_id = cu ? seq_of_row_fp32(cu, n_seqs, i) : 0;
  if (bias_vec) bias = bias_vec[cu ? sq_id * H + bh : bh];
  const size_t kv_base = static_cast<size_t>((bh / H) * H_kv + (bh % H) / (H / H_kv)) * N_k * D;
  float ds_sum = 0.0f;   // this thread's share of sum_j dS_ij
  const size_t base = static_cast<size_t>(bh) * N * D;
  const float slope = slopes ? slopes[bh % H] : 0.0f;
  if (t < D) {
    sq[t] = q[base + static_cast<size_t>(i) * D + t];
    // O = r (P V): the row's factor passes to dO
    sdo[t] = d_o[base + static_cast<size_t>(i) * D + t] * (row_scale ? row_scale[i] : 1.0f);
  }
  __syncthreads();
  const int n_valid = seqlens ? max(0, min(N, seqlens[bh / H])) : N_k;
  int jend = (i >= n_valid && seqlens) ? 0 : min(n_valid, causal ? max(0, min(N_k, i + off + 1)) : N_k);
  const int jbeg = cu ? cu[sq_id] : 0;
  if (cu) jend = min(jend, cu[sq_id + 1]);
  float acc = 0.0f;
  for (int j0 = jbeg; j0 < jend; j0 += kThreads) {
    const int j = j0 + t;
    float ds = 0.0f;
    if (j < jend) {
      const float s = dot_row(sq, k + kv_base + static_cast<size_t>(j) * D, D);
      const float x = fmaf(scale, s, bias) - slope * fabsf(static_cast<float>(i + off - j));
      const float dp = dot_row(sdo, v + kv_base + static_cast<size_t>(j) * D, D);
      ds = sigmoid_slope(x) * dp;
    }
    sds[t] = ds;
    ds_sum += ds;
    __syncthreads();
    if (t < D) {
      const int cnt = min(kThreads, jend - j0);
      for (int jj = 0; jj < cnt; ++jj) acc = fmaf(sds[jj], k[kv_base + static_cast<size_t>(j0 + jj) * D + t], acc);
    }
    __syncthreads();
  }
  if (t < D) dq[base + static_cast<size_t>(i) * D + t] = scale * acc;
  if (dbias) {   // d(bias) of this head: sum of dS over the row, then over the rows (atomics)
    sds[t] = ds_sum;
    __syncthreads();
    for (int half = kThreads / 2; half > 0; half >>= 1) {
      if (t < half) sds[t] += sds[t + half];
      __syncthreads();
    }
    if (t == 0) atomicAdd(dbias + (cu ? sq_id * H + bh : bh), sds[0]);
  }
}

// dV_j = sum_i P_ij dO_i ; dK_j = scale * sum_i dS_ij Q_i, summed over the query heads that read
// this key/value head.  grid (N, B*H_kv), one key row each.
__global__ void bwd_dkdv_fp32_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                     const float* __restrict__ v, const float* __restrict__ d_o,
                                     float* __restrict__ dk, float* __restrict__ dv, int H, int N, int D,
                                     float scale, float bias_scalar, int causal, const float* __restrict__ slopes,
                                     const float* __restrict__ bias_vec, int H_kv, int N_k, int off,
                                     const int* __restrict__ seqlens, const float* __restrict__ row_scale,
                                     const int* __restrict__ cu, int n_seqs) {
  __shared__ float sk[128];
  __shared__ float sv[128];
  __shared__ float sp[kThreads];
  __shared__ float sds[kThreads];
  const int j = blockIdx.x, bh_kv = blockIdx.y, t = threadIdx.x;
  const int group = H / H_kv;
  const size_t kv_base = static_cast<size_t>(bh_kv) * N_k * D;
  if (t < D) {
    sk[t] = k[kv_base + static_cast<size_t>(j) * D + t];
    sv[t] = v[kv_base + static_cast<size_t>(j) * D + t];
  }
  __syncthreads();
  // padded batch: a key past the sequence's length gets zero gradients, queries past it do not count
  const int n_valid = seqlens ? max(0, min(N, seqlens[bh_kv / H_kv])) : N;
  int ibeg = (seqlens && j >= n_valid) ? N : (causal ? max(0, j - off) : 0);
  int iend = n_valid;
  const int sq_id = cu ? seq_of_row_fp32(cu, n_seqs, j) : 0;
  if (cu) {   // batch without padding: queries of the key's own sequence only
    ibeg = max(ibeg, cu[sq_id]);
    iend = cu[sq_id + 1];
  }
  float acc_k = 0.0f, acc_v = 0.0f;
  for (int g = 0; g < group; ++g) {
    const int bh = (bh_kv / H_kv) * H + (bh_kv % H_kv) * group + g;   // query head
    const size_t base = static_cast<size_t>(bh) * N * D;
    const float slope = slopes ? slopes[bh % H] : 0.0f;
    const float bias = bias_vec ? bias_vec[cu ? sq_id * H + bh : bh] : bias_scalar;
    for (int i0 = ibeg; i0 < iend; i0 += kThreads) {
      const int i = i0 + t;
      float p = 0.0f, ds = 0.0f;
      if (i < iend) {
        const float s = dot_row(sk, q + base + static_cast<size_t>(i) * D, D);
        const float x = fmaf(scale, s, bias) - slope * fabsf(static_cast<float>(i + off - j));
        const float r = row_scale ? row_scale[i] : 1.0f;   // O = r (P V): both products see r dO
        p = r * sigmoid_exact(x);
        const float dp = dot_row(sv, d_o + base + static_cast<size_t>(i) * D, D);
        ds = r * sigmoid_slope(x) * dp;
      }
      sp[t] = p;
      sds[t] = ds;
      __syncthreads();
      if (t < D) {
        const int cnt = min(kThreads, iend - i0);
        for (int ii = 0; ii < cnt; ++ii) {
          const size_t row = base + static_cast<size_t>(i0 + ii) * D + t;
          acc_v = fmaf(sp[ii], d_o[row], acc_v);
          acc_k = fmaf(sds[ii], q[row], acc_k);
        }
      }
      __syncthreads();
    }
  }
  if (t < D) {
    dv[kv_base + static_cast<size_t>(j) * D + t] = acc_v;
    dk[kv_base + static_cast<size_t>(j) * D + t] = scale * acc_k;
  }
}

// Row factors of the sequence-length normalisation: n_k^-alpha without a mask, else
// (pos + 1)^-alpha with pos = i + pos0 the query's position (0 for a row that keeps no key).
__global__ void seqlen_norm_kernel(float* __restrict__ out, int N, int N_k, int pos0, int causal, float alpha) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const float count = causal ? static_cast<float>(i + pos0 + 1) : static_cast<float>(N_k);
  out[i] = count >= 1.0f ? powf(count, -alpha) : 0.0f;
}

}  // namespace

int launch_seqlen_norm(float* out, int N, int N_k, int pos0, int causal, float alpha, cudaStream_t stream,
                       unsigned long long* launches, cudaError_t* cuda_err) {
  seqlen_norm_kernel<<<(N + 255) / 256, 256, 0, stream>>>(out, N, N_k, pos0, causal, alpha);
  *launches += 1;
  *cuda_err = cudaGetLastError();
  return *cuda_err == cudaSuccess ? SIGATTN_OK : SIGATTN_ERR_CUDA;
}

int launch_fwd_fp32(const float* q, const float* k, const float* v, float* o, const Problem& p,
                    cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err) {
  dim3 grid(p.N, p.B * p.H);
  fwd_fp32_kernel<<<grid, kThreads, 0, stream>>>(q, k, v, o, p.H, p.N, p.D, p.scale, p.bias, p.causal, p.slopes,
                                                 p.bias_vec, p.kv_heads(), p.key_rows(), p.query_pos0(), p.seqlens,
                                                 p.row_scale, p.cu_seqlens, p.n_seqs);
  *launches += 1;
  *cuda_err = cudaGetLastError();
  return *cuda_err == cudaSuccess ? SIGATTN_OK : SIGATTN_ERR_CUDA;
}

// dtemp[b*H + h] = sum_i <q_i, dq_i> (see the bf16 conversion kernel): one block per (batch, head).
__global__ void __launch_bounds__(256)
dtemp_fp32_kernel(const float* __restrict__ q, const float* __restrict__ dq, size_t per_head, float* __restrict__ dtemp) {
  const size_t base = static_cast<size_t>(blockIdx.x) * per_head;
  double sum = 0.0;
  for (size_t i = threadIdx.x; i < per_head; i += blockDim.x) sum += static_cast<double>(q[base + i]) * dq[base + i];
  __shared__ double part[256];
  part[threadIdx.x] = sum;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if (static_cast<int>(threadIdx.x) < off) part[threadIdx.x] += part[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) dtemp[blockIdx.x] = static_cast<float>(part[0]);
}

int launch_bwd_fp32(const float* q, const float* k, const float* v, const float* d_o, float* dq, float* dk,
                    float* dv, const Problem& p, cudaStream_t stream, unsigned long long* launches,
                    cudaError_t* cuda_err) {
  dim3 grid(p.N, p.B * p.H);
  if (p.dbias) {
    const size_t n_bias = p.cu_seqlens ? static_cast<size_t>(p.n_seqs) * p.H : static_cast<size_t>(p.B) * p.H;
    *cuda_err = cudaMemsetAsync(p.dbias, 0, n_bias * sizeof(float), stream);
    if (*cuda_err != cudaSuccess) return SIGATTN_ERR_CUDA;
  }
  bwd_dq_fp32_kernel<<<grid, kThreads, 0, stream>>>(q, k, v, d_o, dq, p.H, p.N, p.D, p.scale, p.bias, p.causal,
                                                    p.slopes, p.bias_vec, p.dbias, p.kv_heads(), p.key_rows(), p.query_pos0(),
                                                    p.seqlens, p.row_scale, p.cu_seqlens, p.n_seqs);
  dim3 grid_kv(p.key_rows(), p.B * p.kv_heads());
  bwd_dkdv_fp32_kernel<<<grid_kv, kThreads, 0, stream>>>(q, k, v, d_o, dk, dv, p.H, p.N, p.D, p.scale, p.bias,
                                                         p.causal, p.slopes, p.bias_vec, p.kv_heads(), p.key_rows(),
                                                         p.query_pos0(), p.seqlens, p.row_scale, p.cu_seqlens,
                                                         p.n_seqs);
  *launches += 2;
  if (p.dtemp != nullptr) {
    dtemp_fp32_kernel<<<p.B * p.H, 256, 0, stream>>>(q, dq, static_cast<size_t>(p.N) * p.D, p.dtemp);
    *launches += 1;
  }
  *cuda_err = cudaGetLastError();
  return *cuda_err == cudaSuccess ? SIGATTN_OK : SIGATTN_ERR_CUDA;
}

}  // namespace sigattn
