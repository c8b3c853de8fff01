// Fused logits -> sampling transform -> acceptance test -> residual resample / bonus draw
// (Algorithm 1's inner loop, Eq. 5 and Eq. 6), plus the KV commit.  Probability rows q_i never
// reach global memory: each (stream, row) CTA keeps its row in shared memory and leaves only four
// words of statistics; the CTA that finishes last for a stream reduces the accept flags to the
// accepted length k, rebuilds row k on chip and draws the new token.
//
// p = DRAFT distribution, q = TARGET distribution, as in the paper.
#include <math_constants.h>

#include <mutex>

#include "kernels.h"

namespace ssd {

constexpr int SAMP_THREADS = 1024;  // a row of a few thousand logits: short per-thread loops

struct RowStats {
  float zmax;        // max of z = logit / T over the row
  float sum;         // sum of exp(z - zmax) over the kept set
  uint32_t thr_key;  // order-preserving key of the smallest kept value (0 when top-k is off)
  int tie_id_max;    // among values equal to the threshold, ids <= this are kept
};

// Monotone map float -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ bool is_kept(float z, int t, const RowStats& s) {
  uint32_t k = order_key(z);
  return k > s.thr_key || (k == s.thr_key && t <= s.tie_id_max);
}

__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
  for (int i = 1; i < SAMP_THREADS / 32; ++i) r = fmaxf(r, red[i]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ double block_sum_d(double v, double* red) {
  v = warp_sum_d(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double r = 0.0;
  for (int i = 0; i < SAMP_THREADS / 32; ++i) r += red[i];
  __syncthreads();
  return r;
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long r = 0;
  for (int i = 0; i < SAMP_THREADS / 32; ++i) r += red[i];
  __syncthreads();
  return r;
}
// Mass exp(x), x <= 0, in units of 2^-32: integer sums of these do not depend on the order of
// the additions, so the nucleus cut is the same in every run.
__device__ __forceinline__ unsigned long long mass_fx(float x) { return __float2ull_rn(expf(x) * 4294967296.f); }

// Repetition-aware sampling: a nucleus draw that repeats one of the last `win` tokens at least
// win * tau times is thrown away and redrawn from the full softmax.  As one distribution:
//   q(x) = q_nuc(x) [x not repeated] + R q_full(x),  R = mass of q_nuc on the repeated ids.
constexpr int RAS_MAX_WIN = 32;
constexpr int RS_STRIDE = 8;  // floats of row statistics per row: the four of RowStats, sum_full, R
struct Ras {
  int win;               // 0: off
  float thresh;          // win * tau
  const int32_t* recent; // [B, win]: last tokens of T_in, oldest first, pending token last, -1 = none
};
struct RasRow {
  float sum_full;  // sum of exp(z - zmax) over all ids
  float R;
};

struct SampSmem {
  int rep_ids[RAS_MAX_WIN];  // repeated ids of this row's window (-1: none)
  unsigned long long hist_fx[256];
  unsigned long long red_u[SAMP_THREADS / 32];
  unsigned long long mass_above;
  double red_d[SAMP_THREADS / 32];
  double scan[SAMP_THREADS];
  float red_f[SAMP_THREADS / 32];
  int hist[256];
  uint32_t prefix;
  int k_rem, eq_count, tie_id, bad, last, k_acc, y;
};

// Row statistics of the sampling transform: z/T is already in `z` (shared).  Block-collective.
__device__ RowStats compute_row_stats(const float* z, int V, int top_k, float top_p, SampSmem& sm) {
  RowStats st;
  float mx = -CUDART_INF_F;
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) mx = fmaxf(mx, z[t]);
  st.zmax = block_max(mx, sm.red_f);
  st.thr_key = 0u;
  st.tie_id_max = V;
  if (top_k > 0 && top_k < V) {
    // radix select (4 passes of 8 bits, most significant first) of the top_k-th largest key
    if (threadIdx.x == 0) { sm.prefix = 0u; sm.k_rem = top_k; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = threadIdx.x; i < 256; i += SAMP_THREADS) sm.hist[i] = 0;
      __syncthreads();
      const uint32_t prefix = sm.prefix;
      const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
        uint32_t k = order_key(z[t]);
        if ((k & mask) == prefix) atomicAdd(&sm.hist[(k >> shift) & 0xFF], 1);
      }
      __syncthreads();
      if (threadIdx.x < 32) {
        // the highest bin at which the count from the top reaches k_rem (bin 0 if none does), found
        // by the first warp: 8 bins per lane, a suffix sum over the lanes, then a walk of 8 bins
        const int lane = threadIdx.x, rem0 = sm.k_rem;
        int h[8], tot = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { h[i] = sm.hist[8 * lane + i]; tot += h[i]; }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += v;
        }
        const int above = incl - tot;  // in the bins of the higher lanes
        const bool mine = above < rem0 && above + tot >= rem0;
        const unsigned bal = __ballot_sync(0xffffffffu, mine);
        if (bal == 0u ? lane == 0 : mine) {
          int run = above, bin = 8 * lane;  // no crossing: bin 0, everything above it counted
          if (bal == 0u) {
            run = incl - h[0];
          } else {
#pragma unroll
            for (int i = 7; i >= 0; --i) {
              if (run + h[i] >= rem0) { bin = 8 * lane + i; break; }
              run += h[i];
            }
          }
          sm.prefix = prefix | ((uint32_t)bin << shift);
          sm.k_rem = rem0 - run;
          sm.eq_count = sm.hist[bin];
        }
      }
      __syncthreads();
    }
    st.thr_key = sm.prefix;
    if (sm.eq_count > sm.k_rem) {  // equal values straddle the cut: keep the k_rem lowest ids
      if (threadIdx.x == 0) {
        int need = sm.k_rem, t = 0;
        for (; t < V; ++t)
          if (order_key(z[t]) == st.thr_key && --need == 0) break;
        sm.tie_id = t;
      }
      __syncthreads();
      st.tie_id_max = sm.tie_id;
    }
    __syncthreads();
  }
  if (top_p > 0.f && top_p < 1.f) {
    // Nucleus: walking the kept ids from the most to the least probable (lower id first among
    // equals), an id stays while the mass before it is below top_p of the kept mass.  The id at
    // which the running mass first reaches that target is found by a radix select over the
    // ordered keys with histograms of mass instead of counts.
    unsigned long long mine = 0;
    for (int t = threadIdx.x; t < V; t += SAMP_THREADS)
      if (is_kept(z[t], t, st)) mine += mass_fx(z[t] - st.zmax);
    const unsigned long long total = block_sum_u64(mine, sm.red_u);
    const double td = (double)top_p * (double)total;
    unsigned long long target = (unsigned long long)td;
    if ((double)target < td) ++target;  // an id stays iff (mass before it) < target
    if (target < 1) target = 1;
    if (threadIdx.x == 0) { sm.prefix = 0u; sm.mass_above = 0; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = threadIdx.x; i < 256; i += SAMP_THREADS) { sm.hist_fx[i] = 0; sm.hist[i] = 0; }
      __syncthreads();
      const uint32_t prefix = sm.prefix;
      const uint32_t mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
        const uint32_t k = order_key(z[t]);
        if ((k & mask) == prefix && is_kept(z[t], t, st)) {
          atomicAdd(&sm.hist_fx[(k >> shift) & 0xFF], mass_fx(z[t] - st.zmax));
          atomicAdd(&sm.hist[(k >> shift) & 0xFF], 1);
        }
      }
      __syncthreads();
      if (threadIdx.x < 32) {
        // the highest bin at which the mass from the top reaches the target (bin 0 if none does):
        // the same walk as for the counts, on the mass histogram
        const int lane = threadIdx.x;
        const unsigned long long base = sm.mass_above;
        unsigned long long h[8], tot = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { h[i] = sm.hist_fx[8 * lane + i]; tot += h[i]; }
        unsigned long long incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned long long v = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += v;
        }
        const unsigned long long above = base + (incl - tot);
        const bool mine = above < target && above + tot >= target;
        const unsigned bal = __ballot_sync(0xffffffffu, mine);
        if (bal == 0u ? lane == 0 : mine) {
          unsigned long long run = above;
          int bin = 8 * lane;
          if (bal == 0u) {
            run = base + (incl - h[0]);
          } else {
#pragma unroll
            for (int i = 7; i >= 0; --i) {
              if (run + h[i] >= target) { bin = 8 * lane + i; break; }
              run += h[i];
            }
          }
          sm.prefix = prefix | ((uint32_t)bin << shift);
          sm.mass_above = run;
          sm.eq_count = sm.hist[bin];
        }
      }
      __syncthreads();
    }
    const uint32_t cut = sm.prefix;
    int tie_id = st.thr_key == cut ? st.tie_id_max : V;  // ties already trimmed by the top-k cut
    if (threadIdx.x == 0) {
      // ids with the cut's value have equal mass: as many of them as it takes to reach the target
      sm.tie_id = tie_id;
      if (sm.eq_count > 1) {
        unsigned long long each = 0;
        int first = -1;
        for (int t = 0; t < V && first < 0; ++t)
          if (order_key(z[t]) == cut && is_kept(z[t], t, st)) first = t;
        each = first >= 0 ? mass_fx(z[first] - st.zmax) : 1;
        if (each < 1) each = 1;
        unsigned long long need = (target - sm.mass_above + each - 1) / each;
        if (need < 1) need = 1;
        if (need < (unsigned long long)sm.eq_count) {
          int t = first;
          for (; t < V; ++t)
            if (order_key(z[t]) == cut && is_kept(z[t], t, st) && --need == 0) break;
          sm.tie_id = t;
        }
      }
    }
    __syncthreads();
    st.thr_key = cut;
    st.tie_id_max = sm.tie_id;
    __syncthreads();
  }
  double s = 0.0;
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS)
    if (is_kept(z[t], t, st)) s += (double)expf(z[t] - st.zmax);
  st.sum = (float)block_sum_d(s, sm.red_d);
  return st;
}

// Inverse-CDF draw in ascending id over weights w[0..V) (shared): smallest t whose inclusive
// cumulative sum exceeds u * total.  Returns -1 through *total_out <= 0.  Block-collective.
__device__ int block_inverse_cdf(const float* w, int V, float u, SampSmem& sm, double* total_out) {
  const int seg = (V + SAMP_THREADS - 1) / SAMP_THREADS;
  const int t0 = min(threadIdx.x * seg, V), t1 = min(t0 + seg, V);
  double s = 0.0;
  for (int t = t0; t < t1; ++t) s += (double)w[t];
  if (threadIdx.x == 0) sm.y = -1;
  {  // inclusive scan of the threads' sums in a fixed order: inside each warp, then over the warps
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double n = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += n;
    }
    if (lane == 31) sm.red_d[wp] = s;
    __syncthreads();
    if (wp == 0) {
      double v = lane < SAMP_THREADS / 32 ? sm.red_d[lane] : 0.0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const double n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      if (lane < SAMP_THREADS / 32) sm.red_d[lane] = v;
    }
    __syncthreads();
    if (wp > 0) s += sm.red_d[wp - 1];
    sm.scan[threadIdx.x] = s;
  }
  __syncthreads();
  const double total = sm.scan[SAMP_THREADS - 1];
  *total_out = total;
  if (!(total > 0.0)) {
    __syncthreads();
    return -1;
  }
  const double target = (double)u * total;
  const double incl = sm.scan[threadIdx.x];
  const double excl = threadIdx.x == 0 ? 0.0 : sm.scan[threadIdx.x - 1];
  if (excl <= target && target < incl) {
    double run = excl;
    int y = -1;
    for (int t = t0; t < t1; ++t) {
      run += (double)w[t];
      if (w[t] > 0.f) {
        y = t;
        if (run > target) break;
      }
    }
    sm.y = y;
  }
  __syncthreads();
  if (sm.y < 0 && threadIdx.x == 0) {  // u * total rounded up to total: last id with mass
    int t = V - 1;
    while (t > 0 && !(w[t] > 0.f)) --t;
    sm.y = t;
  }
  __syncthreads();
  int y = sm.y;
  __syncthreads();
  return y;
}

// The repeated ids of row r's window: the last `win` tokens of recent[b] ++ x_1..x_r (row r's
// own token x_{r+1} is not part of it).  Block-collective; leaves them in sm.rep_ids.
__device__ void ras_window(const Ras& ras, const int32_t* __restrict__ draft_tokens, int gamma, int b, int r, int V,
                           SampSmem& sm) {
  const int j = threadIdx.x;
  if (j < RAS_MAX_WIN) {
    int rep = -1;
    if (j < ras.win) {
      auto at = [&](int i) {  // i-th token of the window
        const int c = r + i;
        return c < ras.win ? ras.recent[(size_t)b * ras.win + c] : draft_tokens[b * gamma + c - ras.win];
      };
      const int t = at(j);
      if (t >= 0 && t < V) {
        int cnt = 0;
        bool first = true;
        for (int i = 0; i < ras.win; ++i) {
          const bool same = at(i) == t;
          cnt += same;
          if (same && i < j) first = false;
        }
        if (first && (float)cnt >= ras.thresh) rep = t;
      }
    }
    sm.rep_ids[j] = rep;
  }
  __syncthreads();
}
__device__ __forceinline__ bool ras_is_rep(const SampSmem& sm, int win, int t) {
  bool rep = false;
  for (int j = 0; j < win; ++j) rep |= sm.rep_ids[j] == t;
  return rep;
}
// sum_full and R of a row whose nucleus statistics are `st`.  Block-collective.
__device__ RasRow ras_row(const float* z, int V, const RowStats& st, int win, SampSmem& sm) {
  double s = 0.0;
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) s += (double)expf(z[t] - st.zmax);
  RasRow rr;
  rr.sum_full = (float)block_sum_d(s, sm.red_d);
  float R = 0.f;
  for (int j = 0; j < win; ++j) {  // fixed order
    const int t = sm.rep_ids[j];
    if (t >= 0 && is_kept(z[t], t, st)) R += expf(z[t] - st.zmax) / st.sum;
  }
  rr.R = R;
  return rr;
}
// q(t) of the target's sampler: the (top-k, top-p) softmax, or the repetition-aware mixture.
__device__ __forceinline__ float q_value(float zz, int t, const RowStats& st, int win, const RasRow& rr,
                                         const SampSmem& sm) {
  const float e = expf(zz - st.zmax);
  float q = is_kept(zz, t, st) ? e / st.sum : 0.f;
  if (win > 0) {
    if (q > 0.f && ras_is_rep(sm, win, t)) q = 0.f;
    q += rr.R * (e / rr.sum_full);
  }
  return q;
}

// Grid (R, B), R = gamma + 1.
__global__ void __launch_bounds__(SAMP_THREADS)
verify_sampler_kernel(const float* __restrict__ logits, int V,
                      const int32_t* __restrict__ draft_tokens,
                      const float* __restrict__ draft_probs, const float* __restrict__ uniforms,
                      int gamma, float inv_t, int top_k, float top_p, float beta, Ras ras, float* row_stats,
                      int32_t* accept_flags, int32_t* counters, int32_t* __restrict__ accepted_len,
                      int32_t* __restrict__ next_token, int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SampSmem& sm = *reinterpret_cast<SampSmem*>(smem_raw);
  float* z = reinterpret_cast<float*>(smem_raw + sizeof(SampSmem));
  const int r = blockIdx.x, b = blockIdx.y, R = gamma + 1;
  const float* lrow = logits + ((size_t)b * R + r) * V;
  if (threadIdx.x == 0) sm.bad = 0;
  __syncthreads();
  int bad = 0;
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
    float v = lrow[t];
    if (!isfinite(v)) bad = 1;
    z[t] = v * inv_t;
  }
  if (bad) sm.bad = 1;
  __syncthreads();
  if (sm.bad && threadIdx.x == 0) atomicOr(status, SSD_STATUS_NONFINITE);
  RowStats st = compute_row_stats(z, V, top_k, top_p, sm);
  RasRow rr{1.f, 0.f};
  if (ras.win > 0) {
    ras_window(ras, draft_tokens, gamma, b, r, V, sm);
    rr = ras_row(z, V, st, ras.win, sm);
  }
  if (threadIdx.x == 0) {
    int flag = 0;
    if (r < gamma) {  // Eq. 5: accept x_i iff r_i < min(1, q_i(x_i) / p_i(x_i)) + beta
      int x = draft_tokens[b * gamma + r];
      float qx = 0.f, px = 0.f;
      bool valid = true;  // a draft token or probability that cannot be one is rejected, never accepted
      if (x < 0 || x >= V) {
        atomicOr(status, SSD_STATUS_BAD_TOKEN);
        valid = false;
      } else {
        qx = q_value(z[x], x, st, ras.win, rr, sm);
        px = draft_probs[((size_t)b * gamma + r) * V + x];
        if (!(px >= 0.f) || !isfinite(px)) {
          atomicOr(status, SSD_STATUS_BAD_PROB);
          valid = false;
        }
      }
      float ratio = px <= qx ? 1.f : qx / px;
      flag = valid && uniforms[((size_t)b * R + r) * 2] < ratio + beta;
    }
    float* rs = row_stats + ((size_t)b * R + r) * RS_STRIDE;
    rs[0] = st.zmax;
    rs[1] = st.sum;
    rs[2] = __uint_as_float(st.thr_key);
    rs[3] = __int_as_float(st.tie_id_max);
    rs[4] = rr.sum_full;
    rs[5] = rr.R;
    accept_flags[b * R + r] = flag;
    __threadfence();
    int prev = atomicAdd(&counters[b], 1);
    sm.last = prev == R - 1;
  }
  __syncthreads();
  if (!sm.last) return;
  // ---- last CTA of this stream: first rejection, then the one new token ----
  if (threadIdx.x == 0) {
    __threadfence();
    counters[b] = 0;
    int k = gamma;
    for (int i = 0; i < gamma; ++i)
      if (__ldcg(&accept_flags[b * R + i]) == 0) { k = i; break; }
    sm.k_acc = k;
  }
  __syncthreads();
  const int k = sm.k_acc;
  const float* rs = row_stats + ((size_t)b * R + k) * RS_STRIDE;
  RowStats sk;
  sk.zmax = __ldcg(rs + 0);
  sk.sum = __ldcg(rs + 1);
  sk.thr_key = __float_as_uint(__ldcg(rs + 2));
  sk.tie_id_max = __float_as_int(__ldcg(rs + 3));
  const RasRow rk{__ldcg(rs + 4), __ldcg(rs + 5)};
  if (ras.win > 0) ras_window(ras, draft_tokens, gamma, b, k, V, sm);  // row k's repeated ids
  const float* krow = logits + ((size_t)b * R + k) * V;
  const float* prow = k < gamma ? draft_probs + ((size_t)b * gamma + k) * V : nullptr;
  // Eq. 6: w = max(0, q_k - p_k) on a rejection; the bonus row q_{gamma+1} otherwise
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
    float zz = krow[t] * inv_t;
    float q = q_value(zz, t, sk, ras.win, rk, sm);
    z[t] = prow ? fmaxf(0.f, q - prow[t]) : q;
  }
  __syncthreads();
  const float u = uniforms[((size_t)b * R + k) * 2 + 1];
  double total;
  int y = block_inverse_cdf(z, V, u, sm, &total);
  if (y < 0) {  // residual has no mass (numerical corner): draw from q_k itself
    for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
      float zz = krow[t] * inv_t;
      z[t] = q_value(zz, t, sk, ras.win, rk, sm);
    }
    __syncthreads();
    y = block_inverse_cdf(z, V, u, sm, &total);
    if (y < 0) y = 0;
  }
  if (threadIdx.x == 0) {
    accepted_len[b] = k;
    next_token[b] = y;
  }
}

cudaError_t launch_verify_sampler(const float* logits, int V, const int32_t* draft_tokens,
                                  const float* draft_probs, const float* uniforms, int B,
                                  int gamma, float inv_temperature, int top_k, float top_p, float beta,
                                  int ras_window, float ras_tau, const int32_t* recent_tokens,
                                  float* row_stats, int32_t* accept_flags, int32_t* counters,
                                  int32_t* accepted_len, int32_t* next_token, int32_t* status,
                                  cudaStream_t st) {
  Ras ras{0, 0.f, nullptr};
  if (ras_window > 0) {
    if (ras_window > RAS_MAX_WIN || !recent_tokens) return cudaErrorInvalidValue;
    ras = Ras{ras_window, (float)ras_window * ras_tau, recent_tokens};
  }
  size_t smem = sizeof(SampSmem) + (size_t)V * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(verify_sampler_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(gamma + 1, B);
  verify_sampler_kernel<<<grid, SAMP_THREADS, smem, st>>>(
      logits, V, draft_tokens, draft_probs, uniforms, gamma, inv_temperature, top_k, top_p, beta, ras,
      row_stats, accept_flags, counters, accepted_len, next_token, status);
  count_launch();
  return cudaGetLastError();
}

// Draft side (Eq. 2-3): p = transform(logits row), x ~ p by inverse CDF; p is written out in full
// because the verifier needs the whole row (Eq. 6).  One CTA per stream.
__global__ void __launch_bounds__(SAMP_THREADS)
draft_sampler_kernel(const float* __restrict__ logits, int ld_logits, int V,
                     const float* __restrict__ uniform, float inv_t, int top_k, float top_p,
                     int32_t* __restrict__ out_token, int tok_stride, float* __restrict__ out_prob,
                     size_t prob_stride, int32_t* pending, int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SampSmem& sm = *reinterpret_cast<SampSmem*>(smem_raw);
  float* z = reinterpret_cast<float*>(smem_raw + sizeof(SampSmem));
  const int b = blockIdx.x;
  const float* lrow = logits + (size_t)b * ld_logits;
  if (threadIdx.x == 0) sm.bad = 0;
  __syncthreads();
  int bad = 0;
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
    float v = lrow[t];
    if (!isfinite(v)) bad = 1;
    z[t] = v * inv_t;
  }
  if (bad) sm.bad = 1;
  __syncthreads();
  if (sm.bad && threadIdx.x == 0) atomicOr(status, SSD_STATUS_NONFINITE);
  RowStats st = compute_row_stats(z, V, top_k, top_p, sm);
  for (int t = threadIdx.x; t < V; t += SAMP_THREADS) {
    float p = is_kept(z[t], t, st) ? expf(z[t] - st.zmax) / st.sum : 0.f;
    z[t] = p;
    out_prob[(size_t)b * prob_stride + t] = p;
  }
  __syncthreads();
  double total;
  int y = block_inverse_cdf(z, V, uniform[b], sm, &total);
  if (y < 0) y = 0;
  if (threadIdx.x == 0) {
    out_token[(size_t)b * tok_stride] = y;
    pending[b] = y;
  }
}

cudaError_t launch_draft_sampler(const float* logits, int ld_logits, int V, const float* uniform,
                                 int B, float inv_temperature, int top_k, float top_p,
                                 int32_t* out_token, int tok_stride, float* out_prob_row,
                                 size_t prob_stride, int32_t* pending, int32_t* status,
                                 cudaStream_t st) {
  size_t smem = sizeof(SampSmem) + (size_t)V * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(draft_sampler_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  draft_sampler_kernel<<<B, SAMP_THREADS, smem, st>>>(logits, ld_logits, V, uniform,
                                                      inv_temperature, top_k, top_p, out_token, tok_stride,
                                                      out_prob_row, prob_stride, pending, status);
  count_launch();
  return cudaGetLastError();
}

// "Append to T_in" (Algorithm 1): the prefix grows by the k accepted tokens plus the new one.
__global__ void kv_commit_kernel(int32_t* len, int32_t* pending, const int32_t* accepted_len,
                                 const int32_t* next_token, int B, int cap, int max_gamma,
                                 int32_t* status) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int k = accepted_len[b];
  if (k < 0 || k > max_gamma) {  // not an accepted length: the stream stays as it is
    atomicOr(status, SSD_STATUS_BAD_TOKEN);
    return;
  }
  int nl = max(len[b], 0) + 1 + k;
  if (nl > cap) {
    atomicOr(status, SSD_STATUS_KV_OVERFLOW);
    nl = cap;
  }
  len[b] = nl;
  pending[b] = next_token[b];
}

void launch_kv_commit(int32_t* len, int32_t* pending, const int32_t* accepted_len,
                      const int32_t* next_token, int B, int cap, int max_gamma, int32_t* status,
                      cudaStream_t st) {
  kv_commit_kernel<<<(B + 127) / 128, 128, 0, st>>>(len, pending, accepted_len, next_token, B, cap,
                                                    max_gamma, status);
  count_launch();
}

}  // namespace ssd

// ------------------------------------------------------------------------------------------------
// Acceptance step for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code that runs inside a serving loop
// whose memory pool is fixed at start-up, or a plug-in that is handed device pointers by its host
// process and owns none.  ssd_verify needs a workspace such callers cannot provide.  This entry
// point runs the same fused acceptance kernel on logits the caller already has, and keeps the
// kernel's scratch (eight statistics words and one flag per row, one counter per stream, one status
// word) in the fixed device array below instead.
namespace {

constexpr int NOALLOC_MAX_STREAMS = 256;  // streams per call
constexpr int NOALLOC_MAX_ROWS = ssd::R_MAX;  // gamma + 1 <= 16

struct NoAllocScratch {
  float row_stats[NOALLOC_MAX_STREAMS * NOALLOC_MAX_ROWS * ssd::RS_STRIDE];
  int32_t accept_flags[NOALLOC_MAX_STREAMS * NOALLOC_MAX_ROWS];
  int32_t counters[NOALLOC_MAX_STREAMS];
  int32_t status;
};

// About 148 KB, resident on every GPU that loads the library until the process exits.  In host
// code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mu;
NoAllocScratch* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};

// Device address of the scratch array on the current device (looked up once per device).
cudaError_t noalloc_scratch(NoAllocScratch** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = static_cast<NoAllocScratch*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int ssd_accept_noalloc(const float* dev_logits, const int32_t* dev_draft_tokens,
                                  const float* dev_draft_probs, const float* dev_uniforms,
                                  const ssd_verify_params* params, int32_t batch, int32_t vocab,
                                  int32_t* dev_accepted_len, int32_t* dev_next_token,
                                  void* stream) {
  if (!dev_logits || !dev_draft_tokens || !dev_draft_probs || !dev_uniforms || !params ||
      !dev_accepted_len || !dev_next_token)
    return SSD_ERR_NULL;
  if (params->gamma < 1 || params->gamma + 1 > NOALLOC_MAX_ROWS) return SSD_ERR_BAD_GAMMA;
  if (batch < 1 || batch > NOALLOC_MAX_STREAMS) return SSD_ERR_TOO_SMALL;  // beyond the fixed scratch
  if (vocab < 2 || (size_t)vocab * 4 > 180 * 1024) return SSD_ERR_BAD_CONFIG;
  if (!(params->temperature > 0.f) || !isfinite(params->temperature) || !(params->beta >= 0.f) ||
      !isfinite(params->beta))
    return SSD_ERR_BAD_PARAM;
  NoAllocScratch* sc = nullptr;
  cudaError_t e = noalloc_scratch(&sc);
  if (e != cudaSuccess) return ssd::report_cuda_error(e, "ssd_accept_noalloc: cudaGetSymbolAddress");
  cudaStream_t st = (cudaStream_t)stream;
  // the per-stream counters must start at zero; everything else is overwritten before it is read
  e = cudaMemsetAsync(sc->counters, 0, sizeof(int32_t) * (NOALLOC_MAX_STREAMS + 1), st);
  if (e != cudaSuccess) return ssd::report_cuda_error(e, "ssd_accept_noalloc: cudaMemsetAsync");
  e = ssd::launch_verify_sampler(dev_logits, vocab, dev_draft_tokens, dev_draft_probs, dev_uniforms,
                                 batch, params->gamma, 1.0f / params->temperature, params->top_k,
                                 params->top_p, params->beta, params->ras_window, params->ras_tau,
                                 params->dev_recent_tokens, sc->row_stats, sc->accept_flags, sc->counters,
                                 dev_accepted_len, dev_next_token, &sc->status, st);
  if (e != cudaSuccess) return ssd::report_cuda_error(e, "ssd_accept_noalloc: launch");
  return SSD_OK;
}
