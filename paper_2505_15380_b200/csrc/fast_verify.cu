// Launcher of the persistent small-batch verify kernel (the kernel itself: fast_kernel.cuh; its
// variants are instantiated in fast_verify_*.cu).
#include "fast.h"
#include "kernels.h"

namespace ssd {

const void* fast_kernel_r8_split(bool trace);
const void* fast_kernel_r8_bf16(bool trace);
const void* fast_kernel_r16_split(bool trace);
const void* fast_kernel_r16_bf16(bool trace);
const void* fast_kernel_keysplit(bool t16);
size_t fast_misc_bytes();  // per-CTA bookkeeping of the kernel in shared memory

size_t fast_union_bytes(int stage_k, int hd, int T, int o_steps, bool split) {
  const bool t16 = T > 8;
  const size_t step = (size_t)128 * (t16 ? 2 : 1) * (split ? 4 : 2);  // operand bytes per k-step
  size_t af = (size_t)(stage_k / 16) * step;
  size_t red = (size_t)FAST_WARPS * FAST_MAXU * 32 * (t16 ? 16 : 8);
  const int nrow = t16 ? 16 : 8;  // q operand, per-warp K / V tiles (later the partial O), m and l, output operand
  size_t attn = (size_t)(hd / 16) * step + (size_t)FAST_WARPS * 2 * 16 * (hd * 2 + 16) +
                (size_t)FAST_WARPS * nrow * 2 * 4 + (size_t)o_steps * step;
  size_t u = af + red > attn ? af + red : attn;
  return (u + 127) / 128 * 128;
}

cudaError_t launch_fast_forward(const FastParams& p_in, cudaStream_t st) {
  FastParams p = p_in;
  if (p.T < 1 || p.T > FAST_MAX_T || p.m.n_cta > FAST_MAX_CTAS || p.m.max_units > FAST_MAX_UNITS)
    return cudaErrorInvalidValue;
  const size_t uni = fast_union_bytes(p.m.max_stage_k, p.hd, p.T, p.Hq / p.m.o_split * (p.hd / 16), p.split_act != 0);
  const size_t misc = (fast_misc_bytes() + 127) / 128 * 128;
  const size_t max_smem = 227 * 1024;
  if (uni + misc + (size_t)FAST_WARPS * 2 * FAST_SLOT_BYTES > max_smem) return cudaErrorInvalidValue;
  // A shallow ring on purpose: a few KB in flight per warp already saturate HBM, and refill traffic
  // in flight beyond that only queues ahead of the phases' latency-critical loads (3 slots of 5 KB
  // measured best on the 24-layer d = 896 model: 637 us per step against 645 with 4 and 654 with 2).
  int nslot = (int)((max_smem - uni - misc) / ((size_t)FAST_WARPS * FAST_SLOT_BYTES));
  if (nslot > FAST_RING_SLOTS) nslot = FAST_RING_SLOTS;
  p.nslot = nslot;
  p.ring_warp_bytes = nslot * FAST_SLOT_BYTES;
  p.union_off = FAST_WARPS * p.ring_warp_bytes;
  p.misc_off = p.union_off + (int)uni;
  const size_t smem = (size_t)p.misc_off + misc;
  const bool t16 = p.T > 8;
  // the phase trace is a variant of its own: the common path carries no trace code
  const void* kern = p.split_act ? (t16 ? fast_kernel_r16_split(p.trace != nullptr) : fast_kernel_r8_split(p.trace != nullptr))
                                 : (t16 ? fast_kernel_r16_bf16(p.trace != nullptr) : fast_kernel_r8_bf16(p.trace != nullptr));
  // long prefixes: the variant whose CTAs split the keys of a head instead of all walking them
  if (p.key_split && p.split_act && !p.trace && p.attn_part && p.attn_cnt) kern = fast_kernel_keysplit(t16);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  void* args[] = {(void*)&p};
  e = cudaLaunchCooperativeKernel(kern, dim3(p.m.n_cta), dim3(FAST_THREADS), args, smem, st);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
