// ST^3 decode-step attention over a trimmed visual KV cache: sm_100a kernels and the C ABI.
//
// Cache layout (device, caller's workspace).  For every (layer l, sequence b, head h) one block
//   [ K_vis : Nv x D ][ V_vis : Nv x D ][ K_txt : cap x D ][ V_txt : cap x D ]
// with cap = sys_len + max_text_len + max_decode_steps.  The visual rows live in their own
// region so that evicting them never shifts system / text / generated rows; the text region
// holds [S | I | O_1.. ] in order.  ids[l][b][i] is the ORIGINAL visual index of visual row i.
//
// One step = two launches:
//   st3_attend_kernel   one thread block per (l, b, head, row chunk).  The chunk's K and V rows
//                       are brought into shared memory with bulk asynchronous copies
//                       (cp.async.bulk + mbarrier, 16 KB pieces), the block computes the chunk's
//                       logits, its local softmax statistics (m, l) and its un-normalised
//                       output, and - for layers that evict at this step - stores the raw logits
//                       of visual rows.  The block that owns the newest text row also appends it.
//   st3_finish_kernel   one block per (l, b): merges the chunk partials of every head into the
//                       attention output, turns the raw logits into head-summed probabilities
//                       (the visual score alpha), radix-selects the rows to keep (ties toward the
//                       lower original index) and fills the holes among the first n_new rows with
//                       the kept rows of the tail, so the kept rows end up dense and the minimum
//                       number of rows moves.
// The work decomposition is computed on the host from the schedule (row counts are a pure
// function of layer and step), so no table is uploaded per step.
#include "st3.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <new>
#include <vector>

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kFinishThreads = 1024;
constexpr int kMaxChunkRows = 128;  // upper bound on the rows of one work item
constexpr int kMaxLayers = 64;
constexpr int kMaxHeads = 128;
constexpr int kMaxVisual = 8192;
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s: bound on any wait for an async copy

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
  unsigned per_mul[kMaxLayers];     // fast division by (visual + text chunks) of each layer
  unsigned per_shift[kMaxLayers];
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

// ------------------------------------------------------------------------------------------
// Attention (Eq. 2, last row) + raw visual logits + KV append: persistent, warp-specialised
// ------------------------------------------------------------------------------------------
// Two blocks per SM, each with a 3-slot shared-memory ring.  Warp s < 3 is the MANAGER of ring
// slot s: it fetches a work item (layer, sequence, head, row chunk) from a global counter, streams
// the item's K rows, V rows and query into its slot with bulk asynchronous copies, and - once the
// consumers are done with the slot - folds their eight results into the item's partial, refills
// the slot at once and only then stores the partial (plain stores; st3_finish_kernel merges the
// partials of each head).  Warps 3..10 are CONSUMERS in two groups of four that take the slot
// uses alternately (so two items are always being computed); a warp owns a fixed 1/4 of an item's rows
// (K pass: four lanes per row; V pass: a lane owns D/32 output dims and walks the warp's rows):
// logits, tile-local softmax, p.V; the warp leaves its un-normalised result over its own,
// already consumed, K rows.  Loads of the other slots
// are always in flight while one slot is being computed.  Every mbarrier wait is bounded; a
// timeout raises a block-wide abort flag that ends all roles.
constexpr int kConsumers = 8;
constexpr int kGroups = 2;  // consumer warps work in two groups, on two ring slots at a time
constexpr int kGroupWarps = kConsumers / kGroups;
constexpr int kSlots = 3;
constexpr int kAttendThreads = 32 * (kSlots + kConsumers);
constexpr int kQBytes = 512;

struct ItemDesc {
  int nrows;         // < 0: this slot will get no more work
  int want_logits;
  long long glog;    // offset into p.logits of this chunk's first row
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ unsigned fast_div(unsigned n, unsigned mul, unsigned shift) {
  return (__umulhi(n, mul) + n) >> shift;  // exact for n < 2^31 (host: make_fast_div)
}
// Bounded wait of a whole warp that also gives up when another role has already aborted; the
// answer is the same in every lane.
__device__ __forceinline__ bool ring_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  bool ok = mbar_try_wait(bar, parity);
  if (!ok) {
    const long long t0 = clock64();
    while (!(ok = mbar_try_wait(bar, parity))) {
      if (*abort_flag) break;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        atomicOr(status, ST3_DEV_COPY_TIMEOUT);
        break;
      }
    }
  }
  return __all_sync(0xffffffffu, ok);
}

// The finish launch of the previous step may still be running when this kernel starts (programmatic
// dependent launch): visual rows of (l, b) are read only after that launch has signalled them.
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ bool flag_wait(const int* flag, int want, volatile int* abort_flag, int* status) {
  bool ok = ld_acquire(flag) - want >= 0;
  if (!ok) {
    const long long t0 = clock64();
    while (!(ok = ld_acquire(flag) - want >= 0)) {
      __nanosleep(100);
      if (*abort_flag) break;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        atomicOr(status, ST3_DEV_COPY_TIMEOUT);
        break;
      }
    }
  }
  return __all_sync(0xffffffffu, ok);
}

template <typename T, int D>
__global__ void __launch_bounds__(kAttendThreads, 2) st3_attend_kernel(const StepParams p) {
  constexpr int EPL = 16 / sizeof(T);      // elements per 16-byte chunk
  constexpr int ROWB = D * sizeof(T);      // bytes per row
  constexpr int CPL = ROWB / 64;           // 16-byte chunks per lane (a lane owns a quarter row)
  constexpr int kTileBytes = ROWB >= 512 ? 32768 : 16384;  // K (and V) bytes of one ring slot
  constexpr int RMAX = kTileBytes / ROWB;  // rows per item: 64 (128 for 128-byte rows)
  constexpr int TR = RMAX / kGroupWarps;   // rows per consumer warp
  constexpr int GR = TR / 8;               // groups of 8 rows per warp
  constexpr int DPL = D / 32;              // output dims per lane when a warp holds one vector
  constexpr int SLOTB = 2 * kTileBytes + kQBytes;
  static_assert(4 * D <= TR * ROWB, "a warp's result vector must fit its own K rows");
  static_assert(CPL >= 2 && CPL <= 8 && GR >= 1, "unsupported row size");

  extern __shared__ __align__(128) unsigned char smem[];
  // one barrier set per (slot, consumer group): a group sees every phase of its own barriers, so
  // phase parity is never ambiguous
  __shared__ __align__(8) uint64_t s_fullK[kSlots][kGroups], s_fullV[kSlots][kGroups], s_done[kSlots][kGroups];
  __shared__ ItemDesc s_desc[kSlots];
  __shared__ float s_stat[kSlots][kGroupWarps][2];
  __shared__ int s_abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s)
      for (int g = 0; g < kGroups; ++g) {
        mbar_init(&s_fullK[s][g], 1); mbar_init(&s_fullV[s][g], 1); mbar_init(&s_done[s][g], kGroupWarps);
      }
    s_abort = 0;
    mbar_fence_init();
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;
  const int H = p.H;

  if (warp < kSlots) {
    // ===================== manager of slot `warp` =====================
    const int s = warp;
    unsigned char* sK = smem + (size_t)s * SLOTB;
    unsigned char* sV = sK + kTileBytes;
    unsigned char* sQ = sV + kTileBytes;
    const int total = p.total_work;
    constexpr int VPR = ROWB / 16;            // 16-byte vectors per row
    constexpr int LN = VPR <= 16 ? VPR : 16;  // lanes that carry one new row
    constexpr int NV = VPR / LN;              // vectors per such lane

    // A decoded work item, held in registers until its slot is free.
    struct Dec {
      bool valid, has_new;
      int nrows, nbulk, want_logits, wait_for, wait_for_k;
      long long slot, lbh, oidx, oidx_q, glog, lb, lb_k;
      const unsigned char *srcK, *srcV;
      T *newK, *newV;
      uint4 nv[NV];
    };
    int lcur = 0;  // layer of the previous item: this warp's items arrive in increasing order
    long long lb_ready = -1;  // the (l, b) whose visual rows were last seen released by the previous finish launch
    // the first item of every manager is fixed (no round trip to the counter before the first copy);
    // the counter starts behind those and hands out the rest
    int x_next = (int)blockIdx.x * kSlots + s;

    auto decode = [&](Dec& d) {
      const int x = __shfl_sync(0xffffffffu, x_next, 0);
      d.valid = (unsigned)x < (unsigned)total;
      if (!d.valid) return;
      if (lane == 0)  // prefetch the index after this one
        x_next = p.first_dynamic + (int)(atomicAdd(reinterpret_cast<unsigned*>(p.work_counter), 1u) - p.counter_base);
      const int item = (int)fast_div((unsigned)x, p.h_mul, p.h_shift);
      const int h = x - item * H;
      while (lcur + 1 < p.layer_count && item >= p.lstart[lcur + 1]) ++lcur;
      const int l_rel = lcur, l = p.layer_begin + l_rel;
      const int cv = p.cvp[l_rel + 1] - p.cvp[l_rel];
      const int per = cv + p.ct;
      const int off = item - p.lstart[l_rel];
      const int b = (int)fast_div((unsigned)off, p.per_mul[l_rel], p.per_shift[l_rel]);
      const int c = off - b * per;
      const bool is_vis = c < cv;
      int seg_rows, rows_per, ci;
      if (is_vis) {
        seg_rows = p.ncur[l_rel]; rows_per = p.rpv[l_rel]; ci = c;
      } else {
        seg_rows = p.sys_len + __ldg(p.text_len + b) + p.step; rows_per = (seg_rows + p.ct - 1) / p.ct; ci = c - cv;
      }
      const int r0 = ci * rows_per;
      int nrows = min(seg_rows, r0 + rows_per) - r0;
      if (nrows < 0) nrows = 0;
      if (nrows > RMAX) { nrows = RMAX; if (lane == 0) atomicOr(p.status, ST3_DEV_RANGE); }
      d.has_new = !is_vis && p.append && nrows > 0 && r0 + nrows == seg_rows;
      d.nrows = nrows;
      d.nbulk = nrows - (d.has_new ? 1 : 0);
      d.lbh = ((long long)l * p.B + b) * H + h;
      d.oidx = ((long long)l_rel * p.B + b) * H + h;
      // QK heredity (Eq. 6): a lazy layer attends with the query and the keys of its source layer and
      // its own values; the two layers hold the same tokens in the same order
      const int ls = p.lazy_src[l_rel];
      d.oidx_q = ls < 0 ? d.oidx : ((long long)ls * p.B + b) * H + h;
      const long long lbh_k = ls < 0 ? d.lbh : ((long long)(p.layer_begin + ls) * p.B + b) * H + h;
      T* blk = reinterpret_cast<T*>(p.cache) + d.lbh * p.lbh_stride;
      T* blk_k = reinterpret_cast<T*>(p.cache) + lbh_k * p.lbh_stride;
      T* gK = is_vis ? blk_k : blk_k + 2LL * p.Nv * D;
      T* gV = is_vis ? blk + (long long)p.Nv * D : blk + 2LL * p.Nv * D + (long long)p.cap_txt * D;
      d.srcK = reinterpret_cast<const unsigned char*>(gK) + (size_t)r0 * ROWB;
      d.srcV = reinterpret_cast<const unsigned char*>(gV) + (size_t)r0 * ROWB;
      d.want_logits = is_vis && p.ntgt[l_rel] < p.ncur[l_rel] && p.src_layer[l_rel] == l;
      d.lb = (long long)l * p.B + b;
      d.wait_for = is_vis && d.lb != lb_ready ? p.req[l_rel] : 0;
      if (d.wait_for && ld_acquire(p.flags + d.lb) - d.wait_for >= 0) {  // looked up here, off the critical path
        d.wait_for = 0;
        lb_ready = d.lb;
      }
      d.lb_k = (long long)(ls < 0 ? l : p.layer_begin + ls) * p.B + b;
      d.wait_for_k = is_vis && ls >= 0 ? p.req[ls] : 0;  // the source's rows as well
      d.glog = d.lbh * p.Nv + r0;
      d.slot = (long long)item * H + h;
      if (d.has_new) {
        // newest row: fetched from the step's inputs now, stored when the slot is free
        d.newK = ls < 0 ? gK + (long long)(seg_rows - 1) * D : nullptr;  // the source layer stores its own key
        d.newV = gV + (long long)(seg_rows - 1) * D;
        if (lane < 2 * LN) {
          const T* src = lane / LN ? reinterpret_cast<const T*>(p.v_new) + d.oidx * D
                                   : reinterpret_cast<const T*>(p.k_new) + d.oidx_q * D;
#pragma unroll
          for (int i = 0; i < NV; ++i) d.nv[i] = __ldg(reinterpret_cast<const uint4*>(src) + (lane % LN) + i * LN);
        }
      }
    };
    // Starts the copies of a decoded item into this (free) slot.
    auto issue = [&](const Dec& d, int g) {  // g: the consumer group this use of the slot belongs to
      if (d.wait_for) {
        if (!flag_wait(p.flags + d.lb, d.wait_for, abort_flag, p.status)) return;
        lb_ready = d.lb;
      }
      if (d.wait_for_k && !flag_wait(p.flags + d.lb_k, d.wait_for_k, abort_flag, p.status)) return;
      if (d.has_new) {
        if (lane < 2 * LN) {
          const int kv = lane / LN;
#pragma unroll
          for (int i = 0; i < NV; ++i) {
            const int cc = (lane % LN) + i * LN;
            T* dstg = kv ? d.newV : d.newK;
            if (dstg) reinterpret_cast<uint4*>(dstg)[cc] = d.nv[i];
            *reinterpret_cast<uint4*>((kv ? sV : sK) + (size_t)(d.nrows - 1) * ROWB + cc * 16) = d.nv[i];
          }
        }
        __syncwarp();
      }
      if (lane == 0) {
        ItemDesc& sd = s_desc[s];
        sd.nrows = d.nrows; sd.want_logits = d.want_logits; sd.glog = d.glog;
        const uint32_t kb = (uint32_t)d.nbulk * ROWB;
        mbar_expect_tx(&s_fullK[s][g], kb + ROWB);  // K rows + the query (D elements = ROWB bytes)
        bulk_g2s(sQ, reinterpret_cast<const T*>(p.q) + d.oidx_q * D, ROWB, &s_fullK[s][g]);
        if (kb) {
          bulk_g2s(sK, d.srcK, kb, &s_fullK[s][g]);
          mbar_expect_tx(&s_fullV[s][g], kb);
          bulk_g2s(sV, d.srcV, kb, &s_fullV[s][g]);
        } else {
          mbar_arrive(&s_fullV[s][g]);
        }
      }
    };
    Dec cur, nxt;
    decode(cur);
    // Use u of this slot belongs to consumer group (u + s) % kGroups and is that group's (u / kGroups)-th
    // use of the slot, which fixes the parity of the group's barriers.
    if (cur.valid) issue(cur, s % kGroups);
    for (int use = 0; cur.valid; ++use) {
      decode(nxt);  // in the shadow of this item's copies and of the consumers' work
      // ---- wait for this use's consumer group, fold its warps' results ----
      if (!ring_wait(&s_done[s][(use + s) % kGroups], (uint32_t)(use / kGroups) & 1u, abort_flag, p.status)) break;
      const int nw = (cur.nrows + TR - 1) / TR;
      const float mw = lane < nw ? s_stat[s][lane][0] : -INFINITY;
      const float lw = lane < nw ? s_stat[s][lane][1] : 0.f;
      const float M = warp_max(mw);
      const float wgt = lane < nw ? fast_exp2(mw - M) : 0.f;
      const float Lsum = warp_sum(lw * wgt);
      float po[DPL];
#pragma unroll
      for (int j = 0; j < DPL; ++j) po[j] = 0.f;
#pragma unroll
      for (int w = 0; w < kGroupWarps; ++w) {
        const float ww = __shfl_sync(0xffffffffu, wgt, w);
        if (w < nw) {
          const float* res = reinterpret_cast<const float*>(sK + (size_t)w * TR * ROWB) + lane * DPL;  // [D]
#pragma unroll
          for (int j = 0; j < DPL; j += 2) {
            const float2 v2 = *reinterpret_cast<const float2*>(res + j);
            po[j] = fmaf(v2.x, ww, po[j]); po[j + 1] = fmaf(v2.y, ww, po[j + 1]);
          }
        }
      }
      __syncwarp();  // every lane is done reading the slot before it is refilled
      // ---- refill the slot at once ----
      if (nxt.valid) issue(nxt, (use + 1 + s) % kGroups);
      // ---- publish this item's partial (plain stores: the next kernel merges the partials) ----
#pragma unroll
      for (int j = 0; j < DPL; ++j) p.part_acc[cur.slot * D + lane * DPL + j] = po[j];
      if (lane == 0) { p.part_ml[2 * cur.slot] = M; p.part_ml[2 * cur.slot + 1] = Lsum; }
      cur = nxt;
    }
    // out of work (or aborted): an end marker for each consumer group, on the group's own barrier
    if (lane == 0) {
      s_desc[s].nrows = -1;
      for (int g = 0; g < kGroups; ++g) mbar_arrive(&s_fullK[s][g]);
    }
  } else {
    // ===================== consumers =====================
    const int grp = (warp - kSlots) / kGroupWarps;
    const int w = (warp - kSlots) % kGroupWarps;
    const int r8 = lane >> 2, c4 = lane & 3;
    int rot;
    if (CPL == 2) rot = r8 & 1;
    else if (CPL == 4) rot = (c4 >> 1) + 2 * (r8 & 1);
    else rot = lane & 7;
    const float sc = 1.4426950408889634f * rsqrtf((float)D);
    unsigned live = (1u << kSlots) - 1;  // slots that may still deliver work
    for (int round = 0; live; ++round) {
      const int s = round % kSlots;
      const int use = round / kSlots;  // round r is use r / kSlots of slot r % kSlots
      if ((use + s) % kGroups != grp || !(live & (1u << s))) continue;
      const uint32_t par = (uint32_t)(use / kGroups) & 1u;
      if (!ring_wait(&s_fullK[s][grp], par, abort_flag, p.status)) break;
      const int nrows = s_desc[s].nrows;
      if (nrows < 0) { live &= ~(1u << s); continue; }
      const int base = w * TR;
      if (base < nrows) {
        unsigned char* sK = smem + (size_t)s * SLOTB;
        const unsigned char* sV = sK + kTileBytes;
        const unsigned char* sQ = sV + kTileBytes;
        // this lane's quarter of the query, in the rotated chunk order it reads rows in
        u64 q2[CPL][EPL / 2];
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
          const int jj = (j + rot) & (CPL - 1);
          unpack16_pairs(*reinterpret_cast<const uint4*>(sQ + (c4 * CPL + jj) * 16), q2[j]);
        }
        // ---- K pass: four lanes per row, one logit per row ----
        float sl[GR];
        bool ok[GR];
#pragma unroll
        for (int g = 0; g < GR; ++g) {
          const int r = base + g * 8 + r8;
          ok[g] = r < nrows;
          u64 a2[CPL];
#pragma unroll
          for (int j = 0; j < CPL; ++j) a2[j] = 0ull;
          {
            // branch-free: a row past the end re-reads the last valid row and its logit is discarded
            const unsigned char* row = sK + (size_t)min(r, nrows - 1) * ROWB + c4 * (CPL * 16);
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
              const int jj = (j + rot) & (CPL - 1);
              u64 k2[EPL / 2];
              unpack16_pairs(*reinterpret_cast<const uint4*>(row + jj * 16), k2);
#pragma unroll
              for (int e = 0; e < EPL / 2; ++e) fma2(a2[j], q2[j][e], k2[e]);
            }
          }
          float t = 0.f;
#pragma unroll
          for (int j = 0; j < CPL; ++j) t += sum2(a2[j]);
          t += __shfl_xor_sync(0xffffffffu, t, 1);
          t += __shfl_xor_sync(0xffffffffu, t, 2);
          sl[g] = ok[g] ? t * sc : -INFINITY;  // log2-domain logit
        }
        float m = sl[0];
#pragma unroll
        for (int g = 1; g < GR; ++g) m = fmaxf(m, sl[g]);
        m = warp_max(m);
        if (s_desc[s].want_logits && c4 == 0) {
          float* glog = p.logits + s_desc[s].glog;
#pragma unroll
          for (int g = 0; g < GR; ++g)
            if (ok[g]) glog[base + g * 8 + r8] = sl[g];
        }
        float pr[GR], lsum = 0.f;
#pragma unroll
        for (int g = 0; g < GR; ++g) {
          pr[g] = ok[g] ? fast_exp2(sl[g] - m) : 0.f;
          if (c4 == 0) lsum += pr[g];
        }
        lsum = warp_sum(lsum);
        if (!ring_wait(&s_fullV[s][grp], par, abort_flag, p.status)) break;
        // ---- V pass: a lane owns DPL output dims and walks this warp's rows ----
        const int nmine = min(TR, nrows - base);
        u64 acc2[DPL / 2];
#pragma unroll
        for (int i = 0; i < DPL / 2; ++i) acc2[i] = 0ull;
        const unsigned char* vrow = sV + (size_t)base * ROWB + lane * (DPL * (int)sizeof(T));
#pragma unroll
        for (int rr = 0; rr < TR; ++rr) {
          // branch-free: rows past the end carry probability 0 and re-read the last valid row
          const float pv = __shfl_sync(0xffffffffu, pr[rr / 8], (rr % 8) * 4);
          u64 v2[DPL / 2];
          load_pairs<T, DPL>(vrow + (size_t)min(rr, nmine - 1) * ROWB, v2);
          const u64 pp = pack2(pv, pv);
#pragma unroll
          for (int i = 0; i < DPL / 2; ++i) fma2(acc2[i], pp, v2[i]);
        }
        // the warp's un-normalised result [D] goes over its own (consumed) K rows
        float* res = reinterpret_cast<float*>(sK + (size_t)base * ROWB) + lane * DPL;
#pragma unroll
        for (int i = 0; i < DPL / 2; ++i) {
          float lo, hi;
          split2(acc2[i], lo, hi);
          *reinterpret_cast<float2*>(res + 2 * i) = make_float2(lo, hi);
        }
        if (lane == 0) { s_stat[s][w][0] = m; s_stat[s][w][1] = lsum; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_done[s][grp]);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Merge partials, visual scores, top-k (Eq. 3), in-place compaction (Eq. 7's eviction)
// ------------------------------------------------------------------------------------------
// Two blocks per (layer, sequence), on different SMs, that never wait for each other:
//   OUT block   merges the chunk partials of every head into the attention output (a warp per head);
//   TRIM block  merges only the (max, sum) pairs, turns the raw logits into head-summed
//               probabilities, radix-selects the rows to keep, pairs holes with kept tail rows and
//               moves the rows.
// Both are chains of dependent memory round trips, so every phase issues all its loads first.
constexpr int kFinishWarps = kFinishThreads / 32;
constexpr int kHeadBatch = 16;  // logits of one visual row a thread keeps in flight

// (max, 1/sum) of one head's merged softmax from its chunk partials; every lane gets both.
__device__ __forceinline__ void merge_stats(const float2* ml, long long item0, int nit, int H, int h, int lane,
                                            float& M, float& L) {
  float2 v[2];  // the first 64 partials stay in registers
#pragma unroll
  for (int j = 0; j < 2; ++j)
    v[j] = lane + 32 * j < nit ? ml[(item0 + lane + 32 * j) * H + h] : make_float2(-INFINITY, 0.f);
  M = fmaxf(v[0].x, v[1].x);
  for (int i = lane + 64; i < nit; i += 32) M = fmaxf(M, ml[(item0 + i) * H + h].x);
  M = warp_max(M);
  L = v[0].y * fast_exp2(v[0].x - M) + v[1].y * fast_exp2(v[1].x - M);
  for (int i = lane + 64; i < nit; i += 32) {
    const float2 u = ml[(item0 + i) * H + h];
    L += u.y * fast_exp2(u.x - M);
  }
  L = warp_sum(L);
}

template <typename T, int D>
__global__ void __launch_bounds__(kFinishThreads) st3_finish_kernel(const StepParams p) {
  constexpr int ROWB = D * sizeof(T);
  constexpr int VPR = ROWB / 16;  // 16-byte vectors per row
  constexpr int DPL = D / 32;
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ float s_M[kMaxHeads];
  __shared__ float s_invL[kMaxHeads];
  __shared__ int s_hist[256];
  __shared__ int s_scan[kFinishWarps];
  __shared__ float s_half[kFinishThreads / 2];
  __shared__ int s_sel[3];  // digit, count above, count in bin

  // the next step's attention launch may start now; it waits on p.flags for what this launch changes
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int tid = threadIdx.x, lane = tid & 31;
  const int B = p.B, H = p.H, Nv = p.Nv;
  const int units = p.layer_count * B;  // blocks [0, units) trim, blocks [units, 2 units) write the output
  const bool out_role = (int)blockIdx.x >= units;
  const int unit = out_role ? blockIdx.x - units : blockIdx.x;
  const int l_rel = unit / B, b = unit % B;
  const int l = p.layer_begin + l_rel;
  const long long lb = (long long)l * B + b;
  const int nit = p.cvp[l_rel + 1] - p.cvp[l_rel] + p.ct;
  const long long item0 = (long long)p.lstart[l_rel] + (long long)b * nit;
  const float2* ml = reinterpret_cast<const float2*>(p.part_ml);

  if (out_role) {
    if (p.ext_scores) return;  // selection-only launch: nothing to merge yet
    // ===================== OUT block: attention output of every head =====================
    constexpr int kMergeBatch = 8;  // partials in flight per round trip
    for (int h = tid >> 5; h < H; h += kFinishWarps) {
      float a[kMergeBatch][DPL];
      auto load_batch = [&](int i0) {
#pragma unroll
        for (int i = 0; i < kMergeBatch; ++i) {
          if (i0 + i < nit) {
            const float* src = p.part_acc + ((item0 + i0 + i) * H + h) * D + lane * DPL;
            if (DPL == 4) {
              const float4 v = *reinterpret_cast<const float4*>(src);
              a[i][0] = v.x; a[i][1] = v.y; a[i][DPL - 2] = v.z; a[i][DPL - 1] = v.w;
            } else {
              const float2 v = *reinterpret_cast<const float2*>(src);
              a[i][0] = v.x; a[i][DPL - 1] = v.y;
            }
          }
        }
      };
      load_batch(0);
      float M, Lh;
      merge_stats(ml, item0, nit, H, h, lane, M, Lh);
      float o[DPL];
#pragma unroll
      for (int j = 0; j < DPL; ++j) o[j] = 0.f;
      for (int i0 = 0; i0 < nit; i0 += kMergeBatch) {
        if (i0) load_batch(i0);
#pragma unroll
        for (int i = 0; i < kMergeBatch; ++i) {
          if (i0 + i < nit) {
            const float wgt = fast_exp2(ml[(item0 + i0 + i) * H + h].x - M);
#pragma unroll
            for (int j = 0; j < DPL; ++j) o[j] = fmaf(wgt, a[i][j], o[j]);
          }
        }
      }
      const float invL = 1.f / Lh;
      T* out = reinterpret_cast<T*>(p.out) + (((long long)l_rel * B + b) * H + h) * D;
#pragma unroll
      for (int j = 0; j < DPL; ++j) store_out(out + lane * DPL + j, o[j] * invL);
    }
    return;
  }

  // ===================== TRIM block =====================
  const int tt = tid, warp = tid >> 5;
  // Signals that this launch is done with the visual rows, ids and logits of (l, b).
  auto done = [&]() {
    __syncthreads();
    if (tt == 0) { __threadfence(); st_release(p.flags + lb, p.seq); }
  };
  const int n_host = p.ncur[l_rel];
  const int k = min(n_host, p.ntgt[l_rel]);
  const bool evicts = k < n_host;  // same answer in every thread
  const int n_dev = p.n_cur[lb];
  if (!evicts) {
    if (tt == 0) {
      if (n_dev != p.nold[l_rel]) atomicOr(p.status, ST3_DEV_COUNT_MISMATCH);
      else if (n_host != n_dev) p.n_cur[lb] = n_host;  // static-rank cut: only the count changes
    }
    done();
    return;
  }
  int* ids = p.ids + lb * Nv;
  float* mass_by_id = p.mass_by_id + lb * Nv;
  // the scores that decide come from this layer, or from its stage's pruning layer (same rows, same order)
  const int src = p.src_layer[l_rel];
  const long long lb_src = (long long)src * B + b;
  const bool src_here = src >= p.layer_begin && src < p.layer_begin + p.layer_count;
  const float* logits = p.logits_copy[p.src_copy[l_rel]] + lb_src * H * Nv;
  unsigned long long* s_key = reinterpret_cast<unsigned long long*>(smem);  // [Nv]
  int* s_hole = reinterpret_cast<int*>(smem + (size_t)Nv * 8);              // [Nv]
  int* s_mover = s_hole + Nv;                                               // [Nv]
  const int n_cur = n_host;

  // Thread (row r, half g) of a pass sums every second batch of 16 heads of its row; half 1 hands its
  // sum to half 0 through shared memory, so the order of the additions is fixed.  The first batch of
  // the first pass is requested now, together with the (max, sum) pairs: one round trip for both.
  constexpr int kRowsPerPass = kFinishThreads / 2;
  const int ri = tt % kRowsPerPass, hg = tt / kRowsPerPass;
  float pre[kHeadBatch];
  int id0 = 0;
  const bool own_scores = p.ext_scores == nullptr;
  if (own_scores) {
    if (ri < n_cur) {
      if (hg == 0) id0 = ids[ri];
#pragma unroll
      for (int j = 0; j < kHeadBatch; ++j) {
        const int h = hg * kHeadBatch + j;
        pre[j] = h < H ? logits[(long long)h * Nv + ri] : -INFINITY;
      }
    }
    if (src_here) {
      const int ls = src - p.layer_begin;
      const int nit_s = p.cvp[ls + 1] - p.cvp[ls] + p.ct;
      const long long item0_s = (long long)p.lstart[ls] + (long long)b * nit_s;
      for (int h = warp; h < H; h += kFinishWarps) {
        float M, Lh;
        merge_stats(ml, item0_s, nit_s, H, h, lane, M, Lh);
        if (lane == 0) {
          s_M[h] = M; s_invL[h] = 1.f / Lh;
          if (src == l) { p.head_stat[2 * (lb * H + h)] = M; p.head_stat[2 * (lb * H + h) + 1] = 1.f / Lh; }
        }
      }
    } else {  // the pruning layer ran in an earlier launch of this step: its statistics were kept
      for (int h = tt; h < H; h += kFinishThreads) {
        s_M[h] = p.head_stat[2 * (lb_src * H + h)];
        s_invL[h] = p.head_stat[2 * (lb_src * H + h) + 1];
      }
    }
  }
  __syncthreads();
  if (n_dev != n_host) {  // host bookkeeping and device state disagree: flag, do not touch
    if (tt == 0) atomicOr(p.status, ST3_DEV_COUNT_MISMATCH);
    done();
    return;
  }

  // ---- visual scores: probability of every visual row summed over heads ----
  bool bad = false;
  if (!own_scores) {
    // scores supplied by the caller (any finite float): order-preserving map of the bits to unsigned
    const float* ext = p.ext_scores + ((long long)l_rel * B + b) * Nv;
    for (int i = tt; i < n_cur; i += kFinishThreads) {
      const int id = ids[i];
      float sc = ext[id];
      if (!(fabsf(sc) <= 3.0e38f)) { bad = true; sc = -3.0e38f; }
      mass_by_id[id] = sc;
      unsigned u = __float_as_uint(sc);
      u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
      s_key[i] = ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - (unsigned)id);
    }
    __syncthreads();
  }
  for (int i0 = 0; own_scores && i0 < n_cur; i0 += kRowsPerPass) {
    const int i = i0 + ri;
    float pm = 0.f;
    int id = id0;
    if (i < n_cur) {
      if (i0 && hg == 0) id = ids[i];
      for (int h0 = hg * kHeadBatch; h0 < H; h0 += 2 * kHeadBatch) {
        float v[kHeadBatch];
        if (i0 == 0 && h0 == hg * kHeadBatch) {
#pragma unroll
          for (int j = 0; j < kHeadBatch; ++j) v[j] = pre[j];
        } else {
#pragma unroll
          for (int j = 0; j < kHeadBatch; ++j) v[j] = h0 + j < H ? logits[(long long)(h0 + j) * Nv + i] : -INFINITY;
        }
#pragma unroll
        for (int j = 0; j < kHeadBatch; ++j)
          if (h0 + j < H) pm += fast_exp2(v[j] - s_M[h0 + j]) * s_invL[h0 + j];
      }
    }
    if (hg == 1) s_half[ri] = pm;
    __syncthreads();
    if (hg == 0 && i < n_cur) {
      float mass = pm + s_half[ri];
      if (!(mass >= 0.f) || !(mass <= 3.0e38f)) { bad = true; mass = 0.f; }
      mass_by_id[id] = mass;
      s_key[i] = ((unsigned long long)__float_as_uint(mass) << 32) | (unsigned long long)(0xffffffffu - (unsigned)id);
    }
    __syncthreads();
  }
  if (bad) atomicOr(p.status, ST3_DEV_NONFINITE);

  // ---- radix select: the k-th largest 64-bit key (keys are unique: ids are) ----
  unsigned long long prefix = 0ull, mask = 0ull;
  if (k > 0) {
    int need = k;
    for (int shift = 56; shift >= 0; shift -= 8) {
      if (tt < 256) s_hist[tt] = 0;
      __syncthreads();
      for (int i = tt; i < n_cur; i += kFinishThreads) {
        const unsigned long long key = s_key[i];
        if ((key & mask) == prefix) atomicAdd(&s_hist[(int)((key >> shift) & 0xffull)], 1);
      }
      __syncthreads();
      if (warp == 0) {
        int c[8], t = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = s_hist[lane * 8 + j]; t += c[j]; }
        int S = t;  // inclusive suffix sum over lanes (this lane and the higher ones)
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_down_sync(0xffffffffu, S, o);
          if (lane + o < 32) S += v;
        }
        int above = S - t;
        if (above < need && need <= S) {
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (above + c[j] >= need) { s_sel[0] = lane * 8 + j; s_sel[1] = above; s_sel[2] = c[j]; break; }
            above += c[j];
          }
        }
      }
      __syncthreads();
      const int digit = s_sel[0], above = s_sel[1], inbin = s_sel[2];
      need -= above;
      prefix |= (unsigned long long)digit << shift;
      mask |= 0xffull << shift;
      if (need == inbin) break;  // the whole bin is kept: keys >= prefix are exactly the top k
    }
  } else {
    prefix = ~0ull;  // keep nothing (ids are < 2^31, so no key reaches this value)
  }

  if (p.static_rank) {
    // ---- top-index order: the kept row with r larger keys goes to position r, copied from the
    // caller's prompt tensors (the cache rows are only written, so nothing is read after being moved)
    for (int i = tt; i < n_cur; i += kFinishThreads) s_mover[i] = ids[i];
    for (int i = tt; i < n_cur; i += kFinishThreads) {
      const unsigned long long key = s_key[i];
      if (key >= prefix) {
        int r = 0;
        for (int j = 0; j < n_cur; ++j) r += s_key[j] > key;
        s_hole[r] = i;
      }
    }
    __syncthreads();
    unsigned char* blk0 = reinterpret_cast<unsigned char*>(p.cache) + (size_t)(lb * H) * p.lbh_stride * sizeof(T);
    const long long nvec = (long long)k * H * 2 * VPR;
    for (long long v = tt; v < nvec; v += kFinishThreads) {
      const int c = (int)(v % VPR);
      long long r = v / VPR;
      const int kv = (int)(r % 2); r /= 2;
      const int h = (int)(r % H);
      const int j = (int)(r / H);
      const unsigned char* src = reinterpret_cast<const unsigned char*>(kv ? p.v_in : p.k_in) +
                                 ((((size_t)l_rel * B + b) * H + h) * p.t0_max + p.sys_len + s_mover[s_hole[j]]) * ROWB;
      unsigned char* dst = blk0 + (size_t)h * p.lbh_stride * sizeof(T) + (size_t)kv * Nv * ROWB + (size_t)j * ROWB;
      *reinterpret_cast<uint4*>(dst + c * 16) = *reinterpret_cast<const uint4*>(src + c * 16);
    }
    __syncthreads();  // every thread has read the old ids it needs
    for (int j = tt; j < k; j += kFinishThreads) ids[j] = s_mover[s_hole[j]];
    if (tt == 0) p.n_cur[lb] = k;
    done();
    return;
  }

  // ---- pair every hole among the first k rows with a kept row of the tail ----
  const int per = (n_cur + kFinishThreads - 1) / kFinishThreads;
  const int i0 = min(n_cur, tt * per), i1 = min(n_cur, i0 + per);
  int nh = 0, nm = 0;
  for (int i = i0; i < i1; ++i) {
    const bool keep = s_key[i] >= prefix;
    nh += (i < k && !keep);
    nm += (i >= k && keep);
  }
  const int packed = nh | (nm << 16);
  int incl = packed;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_scan[warp] = incl;
  __syncthreads();
  int woff = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kFinishWarps; ++w) {
    if (w < warp) woff += s_scan[w];
    total += s_scan[w];
  }
  const int excl = woff + incl - packed;
  int ph = excl & 0xffff, pm = excl >> 16;
  for (int i = i0; i < i1; ++i) {
    const bool keep = s_key[i] >= prefix;
    if (i < k && !keep) s_hole[ph++] = i;
    if (i >= k && keep) s_mover[pm++] = i;
  }
  __syncthreads();
  const int nmove = total & 0xffff;
  if (nmove != (total >> 16)) {  // cannot happen when exactly k keys pass the threshold
    if (tt == 0) atomicOr(p.status, ST3_DEV_RANGE);
    done();
    return;
  }

  // ---- move the rows (sources are rows >= k, destinations rows < k: disjoint) ----
  const int id_moved = tt < nmove ? ids[s_mover[tt]] : 0;  // in flight together with the rows
  unsigned char* blk0 = reinterpret_cast<unsigned char*>(p.cache) + (size_t)(lb * H) * p.lbh_stride * sizeof(T);
  const long long nvec = (long long)nmove * H * 2 * VPR;
  for (long long v = tt; v < nvec; v += kFinishThreads) {
    const int c = (int)(v % VPR);
    long long r = v / VPR;
    const int kv = (int)(r % 2); r /= 2;
    const int h = (int)(r % H);
    const int j = (int)(r / H);
    unsigned char* base = blk0 + (size_t)h * p.lbh_stride * sizeof(T) + (size_t)kv * Nv * ROWB;
    const uint4 val = *reinterpret_cast<const uint4*>(base + (size_t)s_mover[j] * ROWB + c * 16);
    *reinterpret_cast<uint4*>(base + (size_t)s_hole[j] * ROWB + c * 16) = val;
  }
  if (tt < nmove) ids[s_hole[tt]] = id_moved;
  for (int j = tt + kFinishThreads; j < nmove; j += kFinishThreads) ids[s_hole[j]] = ids[s_mover[j]];
  if (tt == 0) p.n_cur[lb] = k;
  done();
}

// ------------------------------------------------------------------------------------------
// Prompt ingest: rows [S | V | I] of the caller's tensors -> cache regions
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) st3_ingest_kernel(const StepParams p, const T* __restrict__ k,
                                                              const T* __restrict__ v, int t0_max) {
  constexpr int VPR = D * sizeof(T) / 16;
  const int H = p.H, B = p.B, Nv = p.Nv;
  int y = blockIdx.y;
  const int h = y % H; y /= H;
  const int b = y % B;
  const int l_rel = y / B;
  const int l = p.layer_begin + l_rel;
  const int text = __ldg(p.text_len + b);
  const int t0 = p.sys_len + Nv + text;
  const long long lbh_in = ((long long)l_rel * B + b) * H + h;
  const long long lbh = ((long long)l * B + b) * H + h;
  const uint4* srcK = reinterpret_cast<const uint4*>(k + lbh_in * t0_max * D);
  const uint4* srcV = reinterpret_cast<const uint4*>(v + lbh_in * t0_max * D);
  T* blk = reinterpret_cast<T*>(p.cache) + lbh * p.lbh_stride;
  uint4* dKv = reinterpret_cast<uint4*>(blk);
  uint4* dVv = reinterpret_cast<uint4*>(blk + (long long)Nv * D);
  uint4* dKt = reinterpret_cast<uint4*>(blk + 2LL * Nv * D);
  uint4* dVt = reinterpret_cast<uint4*>(blk + 2LL * Nv * D + (long long)p.cap_txt * D);
  const int total = t0 * VPR;
  for (int i = blockIdx.x * kThreads + threadIdx.x; i < total; i += gridDim.x * kThreads) {
    const int row = i / VPR, c = i % VPR;
    const uint4 kk = __ldg(srcK + i), vv = __ldg(srcV + i);
    if (row >= p.sys_len && row < p.sys_len + Nv) {
      const int d = (row - p.sys_len) * VPR + c;
      dKv[d] = kk; dVv[d] = vv;
    } else {
      const int d = (row < p.sys_len ? row : row - Nv) * VPR + c;
      dKt[d] = kk; dVt[d] = vv;
    }
  }
  if (h == 0 && blockIdx.x == 0) {
    const long long lb = (long long)l * B + b;
    for (int i = threadIdx.x; i < Nv; i += kThreads) { p.ids[lb * Nv + i] = i; p.mass_by_id[lb * Nv + i] = 0.f; }
    if (threadIdx.x == 0) p.n_cur[lb] = Nv;
  }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// n / d == (umulhi(n, mul) + n) >> shift for every n < 2^31 (division by an invariant integer).
inline void make_fast_div(unsigned d, unsigned* mul, unsigned* shift) {
  unsigned L = 0;
  while ((1ull << L) < d) ++L;
  *mul = (unsigned)((((1ull << 32) * ((1ull << L) - d)) / d) + 1);
  *shift = L;
}
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

struct Layout {
  size_t elem, cache, part_ml, part_acc, part_ml_bytes, part_acc_bytes, logits, logits_bytes, head_stat, mass, ids, n_cur, flags, text_len, status, stage_q, stage_k, stage_v,
      stage_o, total;
  long long lbh_stride;
  int cap_txt, chunk_rows, max_items;
};

bool valid_config(const st3_config* c) {
  if (!c) return false;
  if (c->num_layers < 1 || c->num_layers > kMaxLayers) return false;
  if (c->num_heads < 1 || c->num_heads > kMaxHeads) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->dtype != ST3_F32 && c->dtype != ST3_BF16) return false;
  if (c->batch < 1 || c->batch > 4096 || c->sys_len < 0 || c->num_visual < 0 || c->num_visual > kMaxVisual)
    return false;
  if (c->max_text_len < 1 || c->max_decode_steps < 0) return false;
  if (c->first_prune_layer < 0 || c->stride < 1) return false;
  if (c->first_ratio_bp < 0 || c->first_ratio_bp > 10000 || c->step_ratio_bp < 0 || c->step_ratio_bp > 10000)
    return false;
  if (c->anneal < ST3_ANNEAL_COSINE || c->anneal > ST3_ANNEAL_EXP) return false;
  if ((c->anneal == ST3_ANNEAL_COSINE || c->anneal == ST3_ANNEAL_LINEAR) && !(c->tau > 0.0)) return false;
  if (c->anneal == ST3_ANNEAL_EXP && !(c->sigma > 0.0)) return false;
  if (c->rows_per_chunk < 0 || c->rows_per_chunk > kMaxChunkRows) return false;
  // lazy layers (QK heredity): the source is the nearest lower layer that is not lazy, and it must hold
  // the same tokens in the same order, i.e. sit in the same pruning stage with stage_shared set
  for (int l = 0; l < c->num_layers; ++l) {
    if (!(c->lazy_mask >> l & 1ull)) continue;
    if (l == 0) return false;
    int sl = l - 1;
    while (sl > 0 && (c->lazy_mask >> sl & 1ull)) --sl;
    if (c->lazy_mask >> sl & 1ull) return false;
    if (c->disable_trim || l < c->first_prune_layer) continue;
    if (!c->stage_shared || sl < c->first_prune_layer) return false;
    if ((l - c->first_prune_layer) / c->stride != (sl - c->first_prune_layer) / c->stride) return false;
  }
  if (c->num_layers < 64 && (c->lazy_mask >> c->num_layers)) return false;
  return true;
}

// Bytes of K (and of V) one ring slot of the attention kernel holds, and the rows that makes.
int tile_bytes(const st3_config* c) {
  const int rowb = c->head_dim * (c->dtype == ST3_BF16 ? 2 : 4);
  return rowb >= 512 ? 32768 : 16384;
}
int tile_rows(const st3_config* c) {
  return tile_bytes(c) / (c->head_dim * (c->dtype == ST3_BF16 ? 2 : 4));
}

int pick_chunk_rows(const st3_config* c) {
  const int cap = tile_rows(c);
  if (c->rows_per_chunk > 0) return c->rows_per_chunk < cap ? c->rows_per_chunk : cap;
  return cap;
}

Layout make_layout(const st3_config* c) {
  Layout L{};
  L.elem = c->dtype == ST3_BF16 ? 2 : 4;
  L.cap_txt = c->sys_len + c->max_text_len + c->max_decode_steps;
  L.chunk_rows = pick_chunk_rows(c);
  L.lbh_stride = 2LL * ((long long)c->num_visual + L.cap_txt) * c->head_dim;
  const size_t lb = (size_t)c->num_layers * c->batch;
  const size_t lbh = lb * c->num_heads;
  L.max_items = (int)(lb * (ceil_div(c->num_visual, L.chunk_rows) + ceil_div(L.cap_txt, L.chunk_rows)));
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.cache = take(lbh * (size_t)L.lbh_stride * L.elem);
  // two copies of the partials: a step's attention launch may run while the previous step's finish
  // launch is still merging
  L.part_ml_bytes = align_up((size_t)L.max_items * c->num_heads * 2 * sizeof(float), 256);
  L.part_acc_bytes = align_up((size_t)L.max_items * c->num_heads * c->head_dim * sizeof(float), 256);
  L.part_ml = take(2 * L.part_ml_bytes);
  L.part_acc = take(2 * L.part_acc_bytes);
  L.logits_bytes = align_up(lbh * (size_t)c->num_visual * sizeof(float), 256);
  L.logits = take(2 * L.logits_bytes);  // two copies, like the partials
  L.head_stat = take(lbh * 2 * sizeof(float));
  L.mass = take(lb * (size_t)c->num_visual * sizeof(float));
  L.ids = take(lb * (size_t)c->num_visual * sizeof(int));
  L.n_cur = take(lb * sizeof(int));
  L.flags = take(lb * sizeof(int));
  L.text_len = take((size_t)c->batch * sizeof(int));
  L.status = take(256);
  const size_t io = lbh * c->head_dim * L.elem;
  L.stage_q = take(io); L.stage_k = take(io); L.stage_v = take(io); L.stage_o = take(io);
  L.total = off;
  return L;
}

double beta_of(const st3_config* c, int t) {
  if (c->anneal == ST3_ANNEAL_NONE || c->disable_trim) return 1.0;
  if (c->anneal == ST3_ANNEAL_EXP) return exp(-(double)t / c->sigma);
  if ((double)t >= c->tau) return 0.0;
  if (c->anneal == ST3_ANNEAL_COSINE) return cos((double)t * M_PI / (2.0 * c->tau));
  return 1.0 - (double)t / c->tau;
}

int count_of(const st3_config* c, int layer, int step) {
  long long keep_bp = 10000;
  if (!c->disable_trim && layer >= c->first_prune_layer) {
    const long long k = (layer - c->first_prune_layer) / c->stride;
    keep_bp = 10000 - c->first_ratio_bp - k * (long long)c->step_ratio_bp;
    if (keep_bp < 0) keep_bp = 0;
  }
  const long long n0 = (long long)c->num_visual * keep_bp / 10000;
  if (layer < c->first_prune_layer || step == 0) return (int)n0;
  return (int)floor((double)n0 * beta_of(c, step) + 1e-9);
}

}  // namespace

struct st3_ctx {
  st3_config cfg;
  Layout lay;
  unsigned char* ws;
  std::vector<int> n_tab;      // [L][max_decode_steps + 1]
  std::vector<int> n_host;     // visual rows each layer holds now (all sequences alike)
  std::vector<int> last_step;  // -1: not prefilled
  std::vector<int> text_len;   // host copy
  bool have_text;
  int max_text;
  cudaStream_t last_stream;
  int64_t launches;
  bool profiling;
  std::vector<cudaEvent_t> ev_pool;  // triples: before attend, after attend, after finish
  size_t ev_used;
  int attend_smem, finish_smem, num_sms, attend_ctas_per_sm;
  int seq;                     // sequence number of the next step's launches (starts at 1)
  unsigned counter_base;       // what the device work counter will read when the next launch starts
  std::vector<int> flag_req;   // per layer: sequence number of the last finish launch over it (0: none)
  std::vector<int> logit_copy; // per layer: which copy holds the logits it wrote last
  std::vector<int> logit_step; // per layer: the step those logits belong to (-1: none)
  bool serialize_next;         // the next attention launch must wait for every earlier launch
};

namespace {

template <typename T, int D>
st3_status launch_step_t(st3_ctx* ctx, const StepParams& p, int total_items, cudaStream_t st, const void* pk,
                         const void* pv, bool ingest, const StepParams* select_first) {
  const st3_config& c = ctx->cfg;
  if (ingest) {
    dim3 grid(8, (unsigned)(c.num_heads * c.batch * p.layer_count));
    st3_ingest_kernel<T, D><<<grid, kThreads, 0, st>>>(p, reinterpret_cast<const T*>(pk),
                                                       reinterpret_cast<const T*>(pv),
                                                       c.sys_len + c.num_visual + c.max_text_len);
    ctx->launches++;
  }
  if (select_first) {  // prune by the caller's scores before the layer attends
    st3_finish_kernel<T, D><<<(unsigned)(2 * p.layer_count * c.batch), kFinishThreads, ctx->finish_smem, st>>>(
        *select_first);
    ctx->launches++;
  }
  cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
  if (ctx->profiling) {
    while (ctx->ev_pool.size() < ctx->ev_used + 3) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return ST3_ERR_CUDA;
      ctx->ev_pool.push_back(e);
    }
    e0 = ctx->ev_pool[ctx->ev_used]; e1 = ctx->ev_pool[ctx->ev_used + 1]; e2 = ctx->ev_pool[ctx->ev_used + 2];
    ctx->ev_used += 3;
    cudaEventRecord(e0, st);
  }
  (void)total_items;
  {
    // Programmatic dependent launch: this launch may start while the previous step's finish launch is
    // still running (that kernel allows it at its start); p.flags orders what the two share.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ctx->num_sms * ctx->attend_ctas_per_sm));
    cfg.blockDim = dim3(kAttendThreads);
    cfg.dynamicSmemBytes = (size_t)ctx->attend_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (ctx->profiling || ingest || ctx->serialize_next) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, st3_attend_kernel<T, D>, p) != cudaSuccess) return ST3_ERR_CUDA;
  }
  if (e1) cudaEventRecord(e1, st);
  st3_finish_kernel<T, D><<<(unsigned)(2 * p.layer_count * c.batch), kFinishThreads, ctx->finish_smem, st>>>(p);
  if (e2) cudaEventRecord(e2, st);
  ctx->launches += 2;
  return cudaGetLastError() == cudaSuccess ? ST3_OK : ST3_ERR_CUDA;
}

template <typename T, int D>
st3_status set_attrs_t(st3_ctx* ctx) {
  if (cudaFuncSetAttribute(st3_attend_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           ctx->attend_smem) != cudaSuccess)
    return ST3_ERR_CUDA;
  if (cudaFuncSetAttribute(st3_finish_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           ctx->finish_smem) != cudaSuccess)
    return ST3_ERR_CUDA;
  return ST3_OK;
}

#define ST3_DISPATCH(ctx, CALL)                                                            \
  ((ctx)->cfg.dtype == ST3_BF16                                                            \
       ? ((ctx)->cfg.head_dim == 128 ? CALL(__nv_bfloat16, 128) : CALL(__nv_bfloat16, 64)) \
       : ((ctx)->cfg.head_dim == 128 ? CALL(float, 128) : CALL(float, 64)))

bool aligned16(const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Common body of prefill (step 0, ingest, no append) and decode (step >= 1, append).
st3_status run_step(st3_ctx* ctx, int step, int layer_begin, int layer_count, const void* q, const void* k,
                    const void* v, void* out, cudaStream_t st, bool prefill, const float* ext_scores = nullptr) {
  const st3_config& c = ctx->cfg;
  const Layout& L = ctx->lay;
  StepParams p;
  memset(&p, 0, sizeof(p));
  p.q = q; p.k_new = prefill ? nullptr : k; p.v_new = prefill ? nullptr : v; p.out = out;
  p.cache = ctx->ws + L.cache;
  p.part_ml = reinterpret_cast<float*>(ctx->ws + L.part_ml + (ctx->seq & 1) * L.part_ml_bytes);
  p.part_acc = reinterpret_cast<float*>(ctx->ws + L.part_acc + (ctx->seq & 1) * L.part_acc_bytes);
  p.flags = reinterpret_cast<int*>(ctx->ws + L.flags);
  p.seq = ctx->seq;
  p.counter_base = ctx->counter_base;
  p.logits = reinterpret_cast<float*>(ctx->ws + L.logits + (ctx->seq & 1) * L.logits_bytes);
  p.logits_copy[0] = reinterpret_cast<const float*>(ctx->ws + L.logits);
  p.logits_copy[1] = reinterpret_cast<const float*>(ctx->ws + L.logits + L.logits_bytes);
  p.head_stat = reinterpret_cast<float*>(ctx->ws + L.head_stat);
  p.mass_by_id = reinterpret_cast<float*>(ctx->ws + L.mass);
  p.ids = reinterpret_cast<int*>(ctx->ws + L.ids);
  p.n_cur = reinterpret_cast<int*>(ctx->ws + L.n_cur);
  p.text_len = reinterpret_cast<const int*>(ctx->ws + L.text_len);
  p.status = reinterpret_cast<int*>(ctx->ws + L.status);
  p.work_counter = p.status + 16;
  p.lbh_stride = L.lbh_stride;
  p.layer_begin = layer_begin; p.layer_count = layer_count; p.B = c.batch; p.H = c.num_heads;
  p.sys_len = c.sys_len; p.Nv = c.num_visual; p.cap_txt = L.cap_txt; p.step = step; p.append = prefill ? 0 : 1;
  p.chunk_rows = L.chunk_rows;
  p.static_rank = c.static_rank ? 1 : 0;
  p.k_in = prefill ? k : nullptr; p.v_in = prefill ? v : nullptr;
  p.t0_max = c.sys_len + c.num_visual + c.max_text_len;
  const int R = L.chunk_rows;
  bool reads_older = false;  // this call's finish launch reads logits an earlier call wrote
  p.ct = ceil_div(c.sys_len + ctx->max_text + step, R);
  p.cvp[0] = 0;
  for (int i = 0; i < layer_count; ++i) {
    const int l = layer_begin + i;
    int ncur = prefill ? c.num_visual : ctx->n_host[l];
    const int tgt = ctx->n_tab[(size_t)l * (c.max_decode_steps + 1) + step];
    if (ext_scores && tgt < ncur) ncur = tgt;  // already pruned by the selection launch when the layer attends
    p.nold[i] = ncur;
    p.req[i] = prefill ? 0 : ctx->flag_req[l];  // prefill follows the ingest launch in stream order
    if (c.static_rank && !prefill && tgt < ncur) ncur = tgt;  // cut first, then attend (Algorithm 3)
    p.ncur[i] = ncur;
    p.ntgt[i] = tgt < ncur ? tgt : ncur;
    p.lazy_src[i] = -1;
    if (c.lazy_mask >> l & 1ull) {
      int sl = l - 1;
      while (sl > 0 && (c.lazy_mask >> sl & 1ull)) --sl;
      if (sl < layer_begin) return ST3_ERR_UNSUPPORTED;  // a lazy layer and its source must share a call
      p.lazy_src[i] = sl - layer_begin;
    }
    // whose scores decide: the layer's own, or (stage-shared) those of its stage's pruning layer
    int src = l;
    if (c.stage_shared && l >= c.first_prune_layer)
      src = c.first_prune_layer + (l - c.first_prune_layer) / c.stride * c.stride;
    p.src_layer[i] = src;
    p.src_copy[i] = ctx->seq & 1;
    if (src < layer_begin) {  // decided in an earlier call of this step
      if (p.ntgt[i] < ncur && !ext_scores && ctx->logit_step[src] != step) return ST3_ERR_BAD_STATE;
      p.src_copy[i] = ctx->logit_copy[src];
      reads_older = true;
    }
    const int cv = ceil_div(ncur, R);
    p.cvp[i + 1] = p.cvp[i] + cv;
    p.lstart[i] = c.batch * (p.cvp[i] + i * p.ct);
    p.rpv[i] = cv ? ceil_div(ncur, cv) : 0;
    make_fast_div((unsigned)(cv + p.ct), &p.per_mul[i], &p.per_shift[i]);
  }
  p.lstart[layer_count] = c.batch * (p.cvp[layer_count] + layer_count * p.ct);
  make_fast_div((unsigned)c.num_heads, &p.h_mul, &p.h_shift);
  const long long total_items = (long long)c.batch * (p.cvp[layer_count] + (long long)layer_count * p.ct);
  if (total_items > L.max_items || total_items * c.num_heads > 0x3fffffffLL) return ST3_ERR_CAPACITY;
  p.total_work = (int)(total_items * c.num_heads);
  p.first_dynamic = ctx->num_sms * ctx->attend_ctas_per_sm * kSlots;

  StepParams psel;
  if (ext_scores) {  // parameters of the selection-only launch: all Nv rows held, cut to the schedule
    psel = p;
    psel.ext_scores = ext_scores;
    for (int i = 0; i < layer_count; ++i) {
      psel.ncur[i] = psel.nold[i] = c.num_visual;
      psel.ntgt[i] = p.ncur[i];
    }
  }
#define ST3_LAUNCH(T, D) launch_step_t<T, D>(ctx, p, (int)total_items, st, k, v, prefill, ext_scores ? &psel : nullptr)
  const st3_status s = ST3_DISPATCH(ctx, ST3_LAUNCH);
#undef ST3_LAUNCH
  if (s != ST3_OK) return s;
  for (int i = 0; i < layer_count; ++i) {
    ctx->n_host[layer_begin + i] = p.ntgt[i];
    ctx->last_step[layer_begin + i] = step;
    ctx->flag_req[layer_begin + i] = ctx->seq;
    if (p.src_layer[i] == layer_begin + i && p.ntgt[i] < p.ncur[i]) {  // it wrote logits in this launch
      ctx->logit_copy[layer_begin + i] = ctx->seq & 1;
      ctx->logit_step[layer_begin + i] = step;
    }
  }
  // Those logits are protected by no flag, so the launch that may overwrite them must not overlap this
  // call's finish launch: it is launched without the programmatic attribute.
  ctx->serialize_next = reads_older;
  ctx->seq++;
  ctx->counter_base += (unsigned)p.total_work;  // one fetch per work item (the first of each manager is fixed)
  ctx->last_stream = st;
  return ST3_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------
extern "C" {

int32_t st3_schedule_count(const st3_config* cfg, int32_t layer, int32_t step) {
  if (!valid_config(cfg) || layer < 0 || layer >= cfg->num_layers || step < 0) return -1;
  return count_of(cfg, layer, step);
}

st3_status st3_workspace_size(const st3_config* cfg, size_t* bytes) {
  if (!valid_config(cfg) || !bytes) return ST3_ERR_INVALID_ARG;
  *bytes = make_layout(cfg).total;
  return ST3_OK;
}

st3_status st3_create(const st3_config* cfg, void* dev_workspace, size_t bytes, st3_ctx** out) {
  if (out) *out = nullptr;
  if (!valid_config(cfg) || !out || !dev_workspace) return ST3_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev_workspace) & 255u) return ST3_ERR_INVALID_ARG;
  const Layout L = make_layout(cfg);
  if (bytes < L.total) return ST3_ERR_WORKSPACE_TOO_SMALL;
  st3_ctx* ctx = new (std::nothrow) st3_ctx();
  if (!ctx) return ST3_ERR_INVALID_ARG;
  ctx->cfg = *cfg;
  ctx->lay = L;
  ctx->ws = static_cast<unsigned char*>(dev_workspace);
  const int T = cfg->max_decode_steps + 1;
  ctx->n_tab.resize((size_t)cfg->num_layers * T);
  for (int l = 0; l < cfg->num_layers; ++l)
    for (int t = 0; t < T; ++t) ctx->n_tab[(size_t)l * T + t] = count_of(cfg, l, t);
  ctx->n_host.assign(cfg->num_layers, cfg->num_visual);
  ctx->last_step.assign(cfg->num_layers, -1);
  ctx->text_len.assign(cfg->batch, 0);
  ctx->have_text = false;
  ctx->max_text = 0;
  ctx->last_stream = nullptr;
  ctx->launches = 0;
  ctx->seq = 1;
  ctx->counter_base = 0;
  ctx->flag_req.assign(cfg->num_layers, 0);
  ctx->logit_copy.assign(cfg->num_layers, 0);
  ctx->logit_step.assign(cfg->num_layers, -1);
  ctx->serialize_next = false;
  ctx->profiling = false;
  ctx->ev_used = 0;
  ctx->attend_smem = kSlots * (2 * tile_bytes(cfg) + kQBytes);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    delete ctx;
    return ST3_ERR_CUDA;
  }
  ctx->num_sms = sms;
  ctx->attend_ctas_per_sm = tile_bytes(cfg) > 16384 ? 1 : 2;
  ctx->finish_smem = (int)((size_t)cfg->num_visual * 16 + 16);
  if (ctx->attend_smem > 200 * 1024 || ctx->finish_smem > 200 * 1024) { delete ctx; return ST3_ERR_UNSUPPORTED; }
#define ST3_ATTR(T, D) set_attrs_t<T, D>(ctx)
  st3_status s = ST3_DISPATCH(ctx, ST3_ATTR);
#undef ST3_ATTR
  if (s == ST3_OK) {
    // bookkeeping area (scores, ids, counts, text lengths, status word) starts cleared
    if (cudaMemsetAsync(ctx->ws + L.mass, 0, L.stage_q - L.mass, nullptr) != cudaSuccess ||
        cudaStreamSynchronize(nullptr) != cudaSuccess)
      s = ST3_ERR_CUDA;
  }
  if (s != ST3_OK) { delete ctx; return s; }
  *out = ctx;
  return ST3_OK;
}

static st3_status prefill_common(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last,
                                 const void* k, const void* v, const int32_t* text_len, const float* scores,
                                 void* out, void* cuda_stream) {
  if (!ctx || !text_len) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c.num_layers) return ST3_ERR_INVALID_ARG;
  if (!aligned16(q_last) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return ST3_ERR_INVALID_ARG;
  int mx = 0;
  for (int b = 0; b < c.batch; ++b) {
    if (text_len[b] < 1) return ST3_ERR_INVALID_ARG;
    if (text_len[b] > c.max_text_len) return ST3_ERR_CAPACITY;
    mx = text_len[b] > mx ? text_len[b] : mx;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  bool changed = !ctx->have_text;
  for (int b = 0; b < c.batch && !changed; ++b) changed = ctx->text_len[b] != text_len[b];
  if (changed) {
    // a new generation: every layer must be prefilled again before it can decode
    for (int b = 0; b < c.batch; ++b) ctx->text_len[b] = text_len[b];
    ctx->max_text = mx;
    ctx->have_text = true;
    for (int l = 0; l < c.num_layers; ++l) ctx->last_step[l] = -1;
    // pageable source: the runtime stages it before returning, so ctx->text_len may change later
    if (cudaMemcpyAsync(ctx->ws + ctx->lay.text_len, ctx->text_len.data(), (size_t)c.batch * sizeof(int),
                        cudaMemcpyHostToDevice, st) != cudaSuccess)
      return ST3_ERR_CUDA;
  }
  return run_step(ctx, 0, layer_begin, layer_count, q_last, k, v, out, st, true, scores);
}

st3_status st3_prefill_select(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last,
                              const void* k, const void* v, const int32_t* text_len, void* out,
                              void* cuda_stream) {
  return prefill_common(ctx, layer_begin, layer_count, q_last, k, v, text_len, nullptr, out, cuda_stream);
}

st3_status st3_prefill_select_scored(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last,
                                     const void* k, const void* v, const int32_t* text_len, const float* scores,
                                     void* out, void* cuda_stream) {
  if (!aligned16(scores)) return ST3_ERR_INVALID_ARG;
  return prefill_common(ctx, layer_begin, layer_count, q_last, k, v, text_len, scores, out, cuda_stream);
}

st3_status st3_decode_step(st3_ctx* ctx, int32_t step, int32_t layer_begin, int32_t layer_count, const void* q,
                           const void* k_new, const void* v_new, void* out, void* cuda_stream) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c.num_layers) return ST3_ERR_INVALID_ARG;
  if (step < 1) return ST3_ERR_INVALID_ARG;
  if (step > c.max_decode_steps) return ST3_ERR_CAPACITY;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return ST3_ERR_INVALID_ARG;
  if (!ctx->have_text) return ST3_ERR_BAD_STATE;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l)
    if (ctx->last_step[l] != step - 1) return ST3_ERR_BAD_STATE;
  return run_step(ctx, step, layer_begin, layer_count, q, k_new, v_new, out, static_cast<cudaStream_t>(cuda_stream),
                  false);
}

st3_status st3_decode_step_host(st3_ctx* ctx, int32_t step, int32_t layer_begin, int32_t layer_count,
                                const void* q_host, const void* k_new_host, const void* v_new_host, void* out_host,
                                void* cuda_stream) {
  if (!ctx || !q_host || !k_new_host || !v_new_host || !out_host) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c.num_layers) return ST3_ERR_INVALID_ARG;
  const Layout& L = ctx->lay;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)layer_count * c.batch * c.num_heads * c.head_dim * L.elem;
  unsigned char* dq = ctx->ws + L.stage_q; unsigned char* dk = ctx->ws + L.stage_k;
  unsigned char* dv = ctx->ws + L.stage_v; unsigned char* dout = ctx->ws + L.stage_o;
  if (cudaMemcpyAsync(dq, q_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(dk, k_new_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(dv, v_new_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return ST3_ERR_CUDA;
  const st3_status s = st3_decode_step(ctx, step, layer_begin, layer_count, dq, dk, dv, dout, cuda_stream);
  if (s != ST3_OK) return s;
  if (cudaMemcpyAsync(out_host, dout, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ST3_ERR_CUDA;
  return ST3_OK;
}

st3_status st3_get_kept(st3_ctx* ctx, int32_t layer, int32_t* ids, int32_t* count, float* mass, void* cuda_stream) {
  if (!ctx || !ids || !count) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  if (layer < 0 || layer >= c.num_layers) return ST3_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Layout& L = ctx->lay;
  const size_t per = (size_t)c.batch * c.num_visual;
  if (per && cudaMemcpyAsync(ids, ctx->ws + L.ids + layer * per * sizeof(int), per * sizeof(int),
                             cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return ST3_ERR_CUDA;
  if (cudaMemcpyAsync(count, ctx->ws + L.n_cur + (size_t)layer * c.batch * sizeof(int), (size_t)c.batch * sizeof(int),
                      cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return ST3_ERR_CUDA;
  if (mass && per && cudaMemcpyAsync(mass, ctx->ws + L.mass + layer * per * sizeof(float), per * sizeof(float),
                                     cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return ST3_ERR_CUDA;
  ctx->last_stream = st;
  return ST3_OK;
}

st3_status st3_get_rows(st3_ctx* ctx, int32_t layer, int32_t b, int32_t h, void* k_vis, void* v_vis, void* k_txt,
                        void* v_txt, void* cuda_stream) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  if (layer < 0 || layer >= c.num_layers || b < 0 || b >= c.batch || h < 0 || h >= c.num_heads)
    return ST3_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Layout& L = ctx->lay;
  const size_t rowb = (size_t)c.head_dim * L.elem;
  const unsigned char* blk =
      ctx->ws + L.cache + (((size_t)layer * c.batch + b) * c.num_heads + h) * (size_t)L.lbh_stride * L.elem;
  const size_t nv = (size_t)c.num_visual * rowb, nt = (size_t)L.cap_txt * rowb;
  void* dst[4] = {k_vis, v_vis, k_txt, v_txt};
  const size_t off[4] = {0, nv, 2 * nv, 2 * nv + nt};
  const size_t len[4] = {nv, nv, nt, nt};
  for (int i = 0; i < 4; ++i)
    if (dst[i] && len[i] &&
        cudaMemcpyAsync(dst[i], blk + off[i], len[i], cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return ST3_ERR_CUDA;
  ctx->last_stream = st;
  return ST3_OK;
}

st3_status st3_get_status(st3_ctx* ctx, int32_t* word) {
  if (!ctx || !word) return ST3_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->last_stream) != cudaSuccess) return ST3_ERR_CUDA;
  int w = 0;
  if (cudaMemcpy(&w, ctx->ws + ctx->lay.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return ST3_ERR_CUDA;
  *word = w;
  return w ? ST3_ERR_DEVICE_CHECK : ST3_OK;
}

st3_status st3_rows_held(st3_ctx* ctx, int64_t* visual_rows, int64_t* other_rows) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  const st3_config& c = ctx->cfg;
  int64_t vis = 0, oth = 0;
  for (int l = 0; l < c.num_layers; ++l) {
    if (ctx->last_step[l] < 0) continue;
    vis += (int64_t)ctx->n_host[l] * c.batch;
    for (int b = 0; b < c.batch; ++b) oth += c.sys_len + ctx->text_len[b] + ctx->last_step[l];
  }
  if (visual_rows) *visual_rows = vis;
  if (other_rows) *other_rows = oth;
  return ST3_OK;
}

st3_status st3_profile_enable(st3_ctx* ctx, int32_t on) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  ctx->profiling = on != 0;
  ctx->ev_used = 0;
  return ST3_OK;
}

st3_status st3_profile_read(st3_ctx* ctx, double* attn_ms, double* finish_ms, int64_t* attn_launches,
                            int64_t* finish_launches) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->last_stream) != cudaSuccess) return ST3_ERR_CUDA;
  double a = 0, f = 0;
  int64_t n = 0;
  for (size_t i = 0; i + 3 <= ctx->ev_used; i += 3) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, ctx->ev_pool[i], ctx->ev_pool[i + 1]) != cudaSuccess) return ST3_ERR_CUDA;
    a += ms;
    if (cudaEventElapsedTime(&ms, ctx->ev_pool[i + 1], ctx->ev_pool[i + 2]) != cudaSuccess) return ST3_ERR_CUDA;
    f += ms;
    ++n;
  }
  ctx->ev_used = 0;
  if (attn_ms) *attn_ms = a;
  if (finish_ms) *finish_ms = f;
  if (attn_launches) *attn_launches = n;
  if (finish_launches) *finish_launches = n;
  return ST3_OK;
}

int64_t st3_launch_count(const st3_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* st3_status_string(st3_status s) {
  switch (s) {
    case ST3_OK: return "ok";
    case ST3_ERR_INVALID_ARG: return "invalid argument";
    case ST3_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case ST3_ERR_BAD_STATE: return "call order violated";
    case ST3_ERR_CAPACITY: return "capacity exceeded";
    case ST3_ERR_CUDA: return "CUDA runtime error";
    case ST3_ERR_DEVICE_CHECK: return "device-side check failed";
    case ST3_ERR_UNSUPPORTED: return "unsupported shape";
  }
  return "unknown status";
}

st3_status st3_destroy(st3_ctx* ctx) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  delete ctx;
  return ST3_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// st3_attend_noalloc: one-shot attention whose split partials live in a static device array
// ------------------------------------------------------------------------------------------
// Some callers cannot hand this library a workspace: code that runs where cudaMalloc is off
// limits (inside a framework's allocator-owned region, in a plugin that was given only its
// input and output tensors, late in a process whose memory is fully committed).  For them the
// chunk partials of the attention go into the fixed array below instead of caller memory.
// The array is part of the loaded module: every GPU that loads the library holds these bytes
// until the process exits, which is why the limit is kept small.
constexpr int kNaChunkRows = 128;
constexpr int kNaMaxSlots = 8192;  // heads x row chunks of one call
constexpr size_t kNaScratchBytes = (size_t)kNaMaxSlots * (2 + 128) * sizeof(float);  // 4 259 840 bytes
static __device__ __align__(256) unsigned char st3_static_scratch[kNaScratchBytes];

namespace {

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) st3_na_partial_kernel(const T* __restrict__ q, const T* __restrict__ K,
                                                                  const T* __restrict__ V, int num_rows, int nchunk,
                                                                  float* part_ml, float* part_acc) {
  constexpr int EPL = 16 / sizeof(T), LPR = D / EPL, RPW = 32 / LPR;
  __shared__ float s_log[kNaChunkRows];
  __shared__ float s_red[kWarps * D];
  __shared__ float s_stat[kWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x, h = blockIdx.y;
  const int r0 = c * kNaChunkRows, nrows = min(num_rows, r0 + kNaChunkRows) - r0;
  const int sub = lane / LPR, lir = lane % LPR;
  const uint4* gK = reinterpret_cast<const uint4*>(K + ((long long)h * num_rows + r0) * D);
  const uint4* gV = reinterpret_cast<const uint4*>(V + ((long long)h * num_rows + r0) * D);
  float qf[EPL];
  unpack16(__ldg(reinterpret_cast<const uint4*>(q + (long long)h * D) + lir), qf);
  const float sc = 1.4426950408889634f * rsqrtf((float)D);
#pragma unroll
  for (int e = 0; e < EPL; ++e) qf[e] *= sc;
  for (int rb = warp * RPW; rb < nrows; rb += kWarps * RPW) {
    const int r = rb + sub;
    float acc = 0.f;
    if (r < nrows) {
      float kf[EPL];
      unpack16(__ldg(gK + (long long)r * LPR + lir), kf);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc = fmaf(qf[e], kf[e], acc);
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (r < nrows && lir == 0) s_log[r] = acc;
  }
  __syncthreads();
  float m = -INFINITY;
  for (int r = tid; r < nrows; r += kThreads) m = fmaxf(m, s_log[r]);
  m = warp_max(m);
  if (lane == 0) s_stat[warp] = m;
  __syncthreads();
  m = s_stat[0];
#pragma unroll
  for (int w = 1; w < kWarps; ++w) m = fmaxf(m, s_stat[w]);
  __syncthreads();
  float lsum = 0.f;
  for (int r = tid; r < nrows; r += kThreads) {
    const float pr = fast_exp2(s_log[r] - m);
    s_log[r] = pr;
    lsum += pr;
  }
  lsum = warp_sum(lsum);
  if (lane == 0) s_stat[warp] = lsum;
  __syncthreads();
  const long long slot = (long long)h * nchunk + c;
  if (tid == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += s_stat[w];
    part_ml[2 * slot] = m;
    part_ml[2 * slot + 1] = t;
  }
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  for (int rb = warp * RPW; rb < nrows; rb += kWarps * RPW) {
    const int r = rb + sub;
    if (r < nrows) {
      float vf[EPL];
      unpack16(__ldg(gV + (long long)r * LPR + lir), vf);
      const float pr = s_log[r];
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pr, vf[e], acc[e]);
    }
  }
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
  }
  if (lane < LPR) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) s_red[warp * D + lir * EPL + e] = acc[e];
  }
  __syncthreads();
  if (tid < D) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += s_red[w * D + tid];
    part_acc[slot * D + tid] = t;
  }
}

template <typename T, int D>
__global__ void st3_na_merge_kernel(T* __restrict__ out, int nchunk, const float* __restrict__ part_ml,
                                    const float* __restrict__ part_acc) {
  const int h = blockIdx.x, d = threadIdx.x;  // D threads
  const long long s0 = (long long)h * nchunk;
  float M = -INFINITY;
  for (int c = 0; c < nchunk; ++c) M = fmaxf(M, part_ml[2 * (s0 + c)]);
  float L = 0.f, o = 0.f;
  for (int c = 0; c < nchunk; ++c) {
    const float w = fast_exp2(part_ml[2 * (s0 + c)] - M);
    L = fmaf(part_ml[2 * (s0 + c) + 1], w, L);
    o = fmaf(part_acc[(s0 + c) * D + d], w, o);
  }
  store_out(out + (long long)h * D + d, o / L);
}

// Device address of st3_static_scratch, looked up once per device.  In host code the array's
// name is only a handle for the runtime, never an address a kernel may be given.
constexpr int kNaMaxDevices = 64;
void* g_na_ptr[kNaMaxDevices] = {nullptr};

st3_status na_scratch(float** ml, float** acc) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return ST3_ERR_CUDA;
  void* p = __atomic_load_n(&g_na_ptr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (cudaGetSymbolAddress(&p, st3_static_scratch) != cudaSuccess || !p) return ST3_ERR_CUDA;
    __atomic_store_n(&g_na_ptr[dev], p, __ATOMIC_RELEASE);  // same value from every racing thread
  }
  *ml = reinterpret_cast<float*>(p);
  *acc = *ml + 2 * (size_t)kNaMaxSlots;
  return ST3_OK;
}

template <typename T, int D>
st3_status na_launch(const void* q, const void* k, const void* v, void* out, int H, int rows, cudaStream_t st) {
  float *ml, *acc;
  const st3_status s = na_scratch(&ml, &acc);
  if (s != ST3_OK) return s;
  const int nchunk = ceil_div(rows, kNaChunkRows);
  st3_na_partial_kernel<T, D><<<dim3((unsigned)nchunk, (unsigned)H), kThreads, 0, st>>>(
      static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), rows, nchunk, ml, acc);
  st3_na_merge_kernel<T, D><<<(unsigned)H, D, 0, st>>>(static_cast<T*>(out), nchunk, ml, acc);
  return cudaGetLastError() == cudaSuccess ? ST3_OK : ST3_ERR_CUDA;
}

}  // namespace

extern "C" st3_status st3_attend_noalloc(const void* q, const void* k, const void* v, void* out, int32_t num_heads,
                                         int32_t num_rows, int32_t head_dim, int32_t dtype, void* cuda_stream) {
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return ST3_ERR_INVALID_ARG;
  if (num_heads < 1 || num_rows < 1 || (head_dim != 64 && head_dim != 128)) return ST3_ERR_INVALID_ARG;
  if (dtype != ST3_F32 && dtype != ST3_BF16) return ST3_ERR_INVALID_ARG;
  // the static array has room for kNaMaxSlots (head, 128-row chunk) partials and no more
  if ((long long)num_heads * ceil_div(num_rows, kNaChunkRows) > kNaMaxSlots) return ST3_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (dtype == ST3_BF16)
    return head_dim == 128 ? na_launch<__nv_bfloat16, 128>(q, k, v, out, num_heads, num_rows, st)
                           : na_launch<__nv_bfloat16, 64>(q, k, v, out, num_heads, num_rows, st);
  return head_dim == 128 ? na_launch<float, 128>(q, k, v, out, num_heads, num_rows, st)
                         : na_launch<float, 64>(q, k, v, out, num_heads, num_rows, st);
}
