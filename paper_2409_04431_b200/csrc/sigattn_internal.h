// Internal interface between the C-ABI layer and the kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace sigattn {

struct Problem {
  int B, H, N, D;
  float scale, bias;
  int causal;
  const float* slopes;    // device pointer to H floats, or nullptr
  const float* bias_vec;  // device pointer to B*H biases that replace `bias`, or nullptr
  float* dbias;           // backward only: device pointer to B*H floats that receive sum dS, or nullptr
  int H_kv;               // heads of k, v (H is a multiple of it; query head h reads head h / (H / H_kv)); 0 = H
  int kv_heads() const { return H_kv > 0 ? H_kv : H; }
  int N_k;                // rows of k, v (N counts the rows of q); 0 = N.  The queries sit at the last N positions.
  int key_rows() const { return N_k > 0 ? N_k : N; }
  int pos0_given;         // 1: `pos0` is the position of query row 0 relative to key row 0 (key/value shards)
  int pos0;               //    0: the queries are the last N positions, pos0 = key_rows() - N
  int query_pos0() const { return pos0_given ? pos0 : key_rows() - N; }
  const int* seqlens;     // device pointer to B valid lengths (padded batch, N_k = N only), or nullptr
  const float* row_scale; // device pointer to N factors, one per query row, applied to O, or nullptr
  float* split_ws;        // forward only: device scratch of B*H*N*D floats that allows splitting the keys of a
                          // head over several thread blocks when there are few queries (decoding), or nullptr
  int acc_only;           // 1 (or 2): accumulate and stop.  Forward: add the partial O, fp32, into split_ws (never cleared,
                          // never converted; o is not written).  Backward: add the partial dQ into the workspace
                          // (not cleared) and leave dq unwritten.  For key/value shards whose results are summed.
                          // 2: the backward also ADDS dK, dV (bf16) into outputs the caller cleared.
  const int* cu_seqlens;  // batch stored without padding (B = 1): device pointer to n_seqs + 1 row offsets, or nullptr;
  int n_seqs;             // bias_vec and dbias then hold one entry per (sequence, head)
  float* dtemp;           // backward only: device pointer to B*H floats that receive sum_i <Q_i, dQ_i>, the gradient
                          // with respect to a temperature t that multiplies the scale as e^t (at t = 0), or nullptr
};

// Every launcher enqueues on `stream`, adds the number of kernels it launched to
// *launches and returns a SIGATTN_* code; on SIGATTN_ERR_CUDA it stores the CUDA error
// in *cuda_err.  `status` is the device-side status word that kernels set when a
// bounded wait expires.

int launch_fwd_fp32(const float* q, const float* k, const float* v, float* o, const Problem& p,
                    cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err);

int launch_bwd_fp32(const float* q, const float* k, const float* v, const float* d_o, float* dq, float* dk,
                    float* dv, const Problem& p, cudaStream_t stream, unsigned long long* launches,
                    cudaError_t* cuda_err);

int launch_fwd_bf16(const void* q, const void* k, const void* v, void* o, const Problem& p, int* status,
                    cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err);

// The forward in its second shape: one query tile per work item, two thread blocks per SM.  Plain problems
// only (self-attention with one key/value head per query head, no padded or unpadded batch, no accumulator).
int launch_fwd_bf16_single(const void* q, const void* k, const void* v, void* o, const Problem& p, int* status,
                           cudaStream_t stream, unsigned long long* launches, cudaError_t* cuda_err);

int launch_bwd_bf16(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk, void* dv,
                    const Problem& p, void* workspace, int* status, cudaStream_t stream,
                    unsigned long long* launches, cudaError_t* cuda_err);

int launch_seqlen_norm(float* out, int N, int N_k, int pos0, int causal, float alpha, cudaStream_t stream,
                       unsigned long long* launches, cudaError_t* cuda_err);

// out (bf16, n elements, n a multiple of 4) = mul * acc (fp32).
int launch_acc_to_bf16(const float* acc, void* out, size_t n, float mul, cudaStream_t stream,
                       unsigned long long* launches, cudaError_t* cuda_err);

size_t bwd_bf16_workspace_bytes(int B, int H, int N, int D);

// Services of the C-ABI layer for entry points that live in other translation units.
// resolve_device: checks that the current device is sm_100 and returns the address of its
// status word (a SIGATTN_* code otherwise).  account: adds to the launch counter and
// remembers the CUDA error behind a SIGATTN_ERR_CUDA for sigattn_last_cuda_error.
int resolve_device(int** status);
void account(unsigned long long launches, int rc, cudaError_t cuda_err);

// Events recorded around the backward's main kernel on the calling thread (nullptr = off).
void set_bwd_timing_events(cudaEvent_t start, cudaEvent_t stop);

}  // namespace sigattn
