// Part of the ST^3 library for sm_100a; included by st3.cu only.
#ifndef ST3_COMMON_CUH_
#define ST3_COMMON_CUH_
#include "st3.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace {


constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kFinishThreads = 1024;
constexpr int kMaxChunkRows = 128;  // upper bound on the rows of one work item
constexpr int kMaxLayers = 64;
constexpr int kMaxHeads = 128;
constexpr int kMaxVisual = 8192;
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s: bound on any wait for an async copy
constexpr int kMaxFollow = 62;  // lazy layers whose values can follow one work item of the layer they inherit from

struct StepParams {
  const void* q;
  const void* k_new;
  const void* v_new;
  void* out;
  void* cache;
  float* part_ml;        // [item*H + h][2]  (m, l) in the log2 domain
  float* part_acc;       // [item*H + h][D]  un-normalised output
  float* logits;         // [l][b][h][Nv]    raw log2-domain logits of visual rows (this step's copy)
  const float* logits_copy[2];  // both copies (a launch writes the one of its sequence parity)
  float* head_stat;      // [l][b][h][2]     (max, 1/sum) of a pruning layer's merged softmax
  float* mass_by_id;     // [l][b][Nv]
  int* ids;              // [l][b][Nv]
  int* n_cur;            // [l][b]
  const int* text_len;   // [b]
  int* status;
  int* work_counter;     // next work item of the running attention launch
  long long lbh_stride;  // elements per (l, b, h) cache block
  int layer_begin, layer_count, B, H;
  int sys_len, Nv, cap_txt, step, append;
  int ct;                   // text chunks per (l, b, h), the same for every sequence
  int chunk_rows;           // rows per work item (<= the kernel's tile capacity)
  int total_work;           // work items x heads of this launch
  int first_dynamic;        // managers of the attention grid: items below this index are pre-assigned
  unsigned counter_base;    // value of the work counter when this launch starts (it is never reset)
  int* flags;               // [l][b] sequence number of the last finish launch that is done with (l, b)
  int seq;                  // sequence number of this step's launches
  int req[kMaxLayers];      // flag value the visual rows of a layer must have reached before they are read
  unsigned h_mul, h_shift;  // fast division by H
  int cvp[kMaxLayers + 1];  // prefix sum of visual chunks per layer (relative layer index)
  int lstart[kMaxLayers + 1];       // first work item of each layer: B * (cvp[l] + l * ct)
  int rpv[kMaxLayers];              // rows per visual chunk of each layer
  unsigned cv_mul[kMaxLayers];      // fast division by the visual chunks of each layer
  unsigned cv_shift[kMaxLayers];
  int text_items;                   // layer_count * B * ct: the attention launch works through these first
  unsigned bct_mul, bct_shift;      // fast division by B * ct
  unsigned ct_mul, ct_shift;        // fast division by ct
  int ncur[kMaxLayers];     // visual rows held before this step (host's schedule bookkeeping)
  int ntgt[kMaxLayers];     // visual rows to hold after this step
  int nold[kMaxLayers];     // visual rows the device should report before this step
  const void* k_in;         // prefill only: the caller's prompt tensors [layer_count][B][H][t0_max][D]
  const void* v_in;
  int t0_max;
  int static_rank;          // 1: keep the kept rows in top-index order, cut them without scoring
  const float* ext_scores;  // prefill with the caller's scores [layer_count][B][Nv]: selection only, no merge
  int src_layer[kMaxLayers];  // the layer whose scores decide this layer's evictions (itself unless stage-shared)
  int src_copy[kMaxLayers];   // which copy of the logits holds that layer's logits
  int lazy_src[kMaxLayers];   // relative index of the layer whose q and K a lazy layer inherits (-1: its own)
  // QK heredity (Eq. 6) without re-reading keys: the lazy layers right above a layer ride on that layer's work
  // items (its probabilities are applied to their value rows as well); they get no items of their own.  The
  // attention launch numbers its work over the remaining ("working") layers only.
  int nwork;                          // working layers of this call
  int wcvp[kMaxLayers + 1];           // prefix sum of their visual chunks
  unsigned char wlayer[kMaxLayers];   // relative layer index of the w-th working layer
  unsigned char nfol[kMaxLayers];     // lazy layers riding on this (working) layer's items
};

// ------------------------------------------------------------------------------------------
// PTX helpers: mbarrier + bulk asynchronous global->shared copy
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 16 bytes -> EPL floats
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8]) {  // bf16 x 8
  f[0] = __uint_as_float(v.x << 16);
  f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16);
  f[3] = __uint_as_float(v.y & 0xffff0000u);
  f[4] = __uint_as_float(v.z << 16);
  f[5] = __uint_as_float(v.z & 0xffff0000u);
  f[6] = __uint_as_float(v.w << 16);
  f[7] = __uint_as_float(v.w & 0xffff0000u);
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4]) {  // f32 x 4
  f[0] = __uint_as_float(v.x);
  f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z);
  f[3] = __uint_as_float(v.w);
}
// Packed pairs of fp32 for fma.rn.f32x2 (two FMAs per issued instruction).
using u64 = unsigned long long;
__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void fma2(u64& d, u64 a, u64 b) { asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b)); }
__device__ __forceinline__ float sum2(u64 v) {
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
  return lo + hi;
}
__device__ __forceinline__ void split2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 bf16x2_pair(unsigned x) {  // two bf16 in one word -> (lo, hi) as fp32
  return pack2(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u));
}
__device__ __forceinline__ void unpack16_pairs(const uint4& v, u64 (&f)[4]) {  // bf16 x 8
  f[0] = bf16x2_pair(v.x); f[1] = bf16x2_pair(v.y); f[2] = bf16x2_pair(v.z); f[3] = bf16x2_pair(v.w);
}
__device__ __forceinline__ void unpack16_pairs(const uint4& v, u64 (&f)[2]) {  // f32 x 4
  f[0] = pack2(__uint_as_float(v.x), __uint_as_float(v.y));
  f[1] = pack2(__uint_as_float(v.z), __uint_as_float(v.w));
}
// DPL consecutive elements of a row, as DPL/2 packed fp32 pairs
template <typename T, int DPL>
__device__ __forceinline__ void load_pairs(const unsigned char* p, u64 (&f)[DPL / 2]) {
  if constexpr (sizeof(T) == 2 && DPL == 4) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    f[0] = bf16x2_pair(v.x); f[DPL / 2 - 1] = bf16x2_pair(v.y);
  } else if constexpr (sizeof(T) == 2) {
    f[0] = bf16x2_pair(*reinterpret_cast<const unsigned*>(p));
  } else if constexpr (DPL == 4) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = pack2(v.x, v.y); f[DPL / 2 - 1] = pack2(v.z, v.w);
  } else {
    const float2 v = *reinterpret_cast<const float2*>(p);
    f[0] = pack2(v.x, v.y);
  }
}
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}


}  // namespace

#endif  // ST3_COMMON_CUH_
