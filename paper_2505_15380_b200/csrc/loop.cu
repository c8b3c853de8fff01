// Bookkeeping of the device-resident SSD iteration (Algorithm 1's loop body without a host round
// trip): which uniforms an iteration consumes, and what "append to T_in" means for the draft
// model's cache and for the emitted token stream.
#include "kernels.h"

namespace ssd {

// Row `iteration % n_rows` of the caller's pool of uniforms, float [n_rows][B][gamma + 2 (gamma + 1)]
// (per stream: gamma draws for x_i ~ p_i, then the (r_i, u_i) pairs of the gamma + 1 verify rows),
// is spread into the layouts the kernels read: draft_uni [gamma][B], verify_uni [B][gamma + 1][2].
__global__ void loop_stage_uniforms_kernel(const float* __restrict__ pool, int n_rows,
                                           const int32_t* __restrict__ iteration, int B, int gamma,
                                           float* __restrict__ draft_uni, float* __restrict__ verify_uni) {
  const int per = gamma + 2 * (gamma + 1);
  const int it = ((*iteration % n_rows) + n_rows) % n_rows;
  const float* row = pool + (size_t)it * B * per;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B * per; i += gridDim.x * blockDim.x) {
    const int b = i / per, j = i % per;
    if (j < gamma) draft_uni[j * B + b] = row[i];
    else verify_uni[(size_t)b * 2 * (gamma + 1) + (j - gamma)] = row[i];
  }
}

void launch_loop_stage_uniforms(const float* pool, int n_rows, const int32_t* iteration, int B, int gamma,
                                float* draft_uni, float* verify_uni, cudaStream_t st) {
  const int n = B * (gamma + 2 * (gamma + 1));
  loop_stage_uniforms_kernel<<<(n + 255) / 256, 256, 0, st>>>(pool, n_rows, iteration, B, gamma, draft_uni,
                                                             verify_uni);
  count_launch();
}

// End of an iteration, per stream: the prefix grew by x_1..x_k and the new token y.
//  * emitted tokens: x_1..x_k, y are appended to the stream's output (as far as it has room);
//  * draft cache: the gamma draft steps left K/V for the old pending token and x_1..x_{gamma-1}.
//    The next iteration's first draft step always feeds two ids, [token before y, y], at the
//    position of the first: len -= gamma - k.  After a full acceptance that computes the missing
//    K/V of x_gamma; otherwise it recomputes one cached row with the same inputs.  One rule for
//    every stream, so a batch needs no host decision;
//  * in_ids[b] = [k > 0 ? x_k : the token that was pending, y].
__global__ void loop_finish_kernel(int32_t* draft_len, int32_t* draft_pending, int cap, int32_t* in_ids,
                                   const int32_t* __restrict__ draft_tokens, int gamma,
                                   const int32_t* __restrict__ accepted_len,
                                   const int32_t* __restrict__ next_token, int B, int32_t* out_tokens,
                                   int out_capacity, int32_t* out_count, int32_t* accept_log, int n_rows,
                                   int32_t* iteration, int32_t* recent, int win, int32_t* status) {
  const int it = ((*iteration % n_rows) + n_rows) % n_rows;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {  // launched as one block
    int k = accepted_len[b];
    if (k < 0 || k > gamma) {  // not an accepted length: emit nothing, keep the draft where it is
      atomicOr(status, SSD_STATUS_BAD_TOKEN);
      k = -1;
    }
    if (accept_log) accept_log[(size_t)it * B + b] = k;
    if (k >= 0) {
      const int y = next_token[b];
      int n = out_count[b];
      for (int i = 0; i <= k; ++i) {
        if (n < out_capacity) out_tokens[(size_t)b * out_capacity + n] = i < k ? draft_tokens[b * gamma + i] : y;
        ++n;
      }
      out_count[b] = n;
      if (recent) {  // the window of the repetition-aware sampler: the last `win` tokens of T_in
        const int e = k + 1;
        for (int i = 0; i < win; ++i) {  // in place: entry i takes a value from at or beyond i
          const int src = i + e;
          recent[(size_t)b * win + i] = src < win ? recent[(size_t)b * win + src]
                                                  : (src - win < k ? draft_tokens[b * gamma + src - win] : y);
        }
      }
      const int prev = k > 0 ? draft_tokens[b * gamma + k - 1] : in_ids[2 * b + 1];
      in_ids[2 * b] = prev;
      in_ids[2 * b + 1] = y;
      draft_len[b] = min(max(draft_len[b] - (gamma - k), 0), cap);
      draft_pending[b] = y;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) *iteration = *iteration + 1;
}

void launch_loop_finish(int32_t* draft_len, int32_t* draft_pending, int cap, int32_t* in_ids,
                        const int32_t* draft_tokens, int gamma, const int32_t* accepted_len,
                        const int32_t* next_token, int B, int32_t* out_tokens, int out_capacity,
                        int32_t* out_count, int32_t* accept_log, int n_rows, int32_t* iteration,
                        int32_t* recent_tokens, int ras_window, int32_t* status, cudaStream_t st) {
  // one block: every thread reads the iteration counter before the last thread advances it
  loop_finish_kernel<<<1, 1024, 0, st>>>(draft_len, draft_pending, cap, in_ids, draft_tokens, gamma, accepted_len,
                                         next_token, B, out_tokens, out_capacity, out_count, accept_log, n_rows,
                                         iteration, recent_tokens, ras_window, status);
  count_launch();
}

}  // namespace ssd
