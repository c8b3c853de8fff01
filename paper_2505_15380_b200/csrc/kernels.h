// Host-side launchers of the kernels (one translation unit per kernel family).
#pragma once
#include "common.cuh"

namespace ssd {

// Process-wide count of kernels enqueued by the launchers below.
void count_launch(int n = 1);
uint64_t launch_count();
// Records a CUDA error for ssd_last_cuda_error and returns SSD_ERR_CUDA (api.cu).
int report_cuda_error(cudaError_t e, const char* what);

enum Epilogue { EPI_STORE_F32 = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2 };

// elementwise.cu
void launch_gather_verify_ids(const int32_t* pending, const int32_t* draft_tokens, int gamma,
                              int B, int32_t* row_ids, cudaStream_t st);
void launch_embed(int dtype, const void* table, int vocab_in, int d, const int32_t* row_ids, int M,
                  float* h, int32_t* status, cudaStream_t st);
void launch_rope_table(const int32_t* len, RowMap rm, const double* inv_freq, int half, float* cs,
                       cudaStream_t st);
void launch_rmsnorm(int dtype, const float* h, const void* gain, float* out, int M, int d, float eps,
                    cudaStream_t st);
void launch_qkv_post(int dtype, const float* qkv, const float* cs, float* qrot, void* kv_layer,
                     const int32_t* len, RowMap rm, int cap, int Hq, int Hkv, int hd,
                     int32_t* status, cudaStream_t st);
void launch_advance_len(int32_t* len, int32_t* pending, int b, int add, const int32_t* ids,
                        int pending_index, cudaStream_t st);

void launch_kv_restore(int32_t* len, int32_t* pending, const int32_t* src_len,
                       const int32_t* src_pending, int B, int cap, cudaStream_t st);
void launch_advance_all(int32_t* len, int B, int add, int cap, int32_t* status, cudaStream_t st);

// gemm_simt.cu :  C[M,N] = A[M,K] * W[N,K]^T with a fused epilogue
//   EPI_STORE_F32 : C[m, n]   = acc + bias[n]                       (bias may be null)
//   EPI_RESIDUAL  : C[m, n]  += acc
//   EPI_SWIGLU    : C[m, n/2] = silu(acc[2j]) * acc[2j+1]           (W rows interleaved g,u)
// Activations and outputs are fp32; `dtype` is the storage type of W and bias.
cudaError_t launch_gemm_simt(int dtype, int epi, const float* A, int lda, const void* W,
                             const void* bias, float* C, int ldc, int M, int N, int K,
                             cudaStream_t st);

// attention_simt.cu
cudaError_t launch_attention_simt(int dtype, const float* qrot, const void* kv_layer,
                                  const int32_t* len, RowMap rm, int cap, int Hq, int Hkv, int hd,
                                  float* part, int nsplit_max, float* out, cudaStream_t st);

// sampler.cu
cudaError_t launch_verify_sampler(const float* logits, int V, const int32_t* draft_tokens,
                                  const float* draft_probs, const float* uniforms, int B,
                                  int gamma, float inv_temperature, int top_k, float top_p, float beta,
                                  int ras_window, float ras_tau, const int32_t* recent_tokens,
                                  float* row_stats, int32_t* accept_flags, int32_t* counters,
                                  int32_t* accepted_len, int32_t* next_token, int32_t* status,
                                  cudaStream_t st);
// out_token[b * tok_stride] and out_prob_row[b * prob_stride + t]: the strides let a loop write
// step i of every stream straight into the [B, gamma] / [B, gamma, V] arrays the verifier reads.
cudaError_t launch_draft_sampler(const float* logits, int ld_logits, int V, const float* uniform,
                                 int B, float inv_temperature, int top_k, float top_p,
                                 int32_t* out_token, int tok_stride, float* out_prob_row,
                                 size_t prob_stride, int32_t* pending, int32_t* status,
                                 cudaStream_t st);

// loop.cu: bookkeeping kernels of the device-resident SSD iteration
void launch_loop_stage_uniforms(const float* pool, int n_rows, const int32_t* iteration, int B, int gamma,
                                float* draft_uni, float* verify_uni, cudaStream_t st);
void launch_loop_finish(int32_t* draft_len, int32_t* draft_pending, int cap, int32_t* in_ids,
                        const int32_t* draft_tokens, int gamma, const int32_t* accepted_len,
                        const int32_t* next_token, int B, int32_t* out_tokens, int out_capacity,
                        int32_t* out_count, int32_t* accept_log, int n_rows, int32_t* iteration,
                        int32_t* recent_tokens, int ras_window, int32_t* status, cudaStream_t st);
void launch_kv_commit(int32_t* len, int32_t* pending, const int32_t* accepted_len,
                      const int32_t* next_token, int B, int cap, int max_gamma, int32_t* status,
                      cudaStream_t st);

}  // namespace ssd
