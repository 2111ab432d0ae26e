// Part of the ST^3 library for sm_100a; included by st3.cu only.
#ifndef ST3_ATTEND_CUH_
#define ST3_ATTEND_CUH_
#include "st3_common.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// Attention (Eq. 2, last row) + raw visual logits + KV append: persistent, warp-specialised
// ------------------------------------------------------------------------------------------
// Two blocks per SM, each with a 3-slot shared-memory ring.  Warp s < 3 is the MANAGER of ring
// slot s: it fetches a work item (layer, sequence, head, row chunk) from a global counter, streams
// the item's K rows, V rows and query into its slot with bulk asynchronous copies, and - once the
// consumers are done with the slot - folds their four results into the item's partial, refills
// the slot at once and only then stores the partial (plain stores; st3_finish_kernel merges the
// partials of each head).  Warps 3..10 are CONSUMERS in two groups of four that take the slot
// uses alternately (so two items are always being computed); a warp owns a fixed 1/4 of an item's rows
// (K pass: four lanes per row; V pass: a lane owns D/32 output dims and walks the warp's rows):
// logits, tile-local softmax, p.V; the warp leaves its un-normalised result over its own,
// already consumed, K rows.  Loads of the other slots are always in flight while one slot is
// being computed.  Every mbarrier wait is bounded; a
// timeout raises a block-wide abort flag that ends all roles.
//
// QK heredity (Eq. 6): an item of a layer with lazy layers above it is followed, in the same ring slot, by
// value-only uses: the consumers of the item leave its probabilities in shared memory, and each following use
// of the slot brings the value rows of the same chunk of up to two lazy layers (one per tile area), which the
// next consumer group multiplies with those probabilities.  A lazy layer's keys are never read and it has no
// work items of its own; a value-only use moves as many bytes as a plain item and takes the same time.
constexpr int kConsumers = 8;
constexpr int kGroups = 2;  // consumer warps work in two groups, on two ring slots at a time
constexpr int kGroupWarps = kConsumers / kGroups;
constexpr int kSlots = 3;
constexpr int kAttendThreads = 32 * (kSlots + kConsumers);
constexpr int kQBytes = 512;

// What the consumers need to know of a use of a ring slot, packed so that one shared-memory load brings it.
struct ItemDesc {
  int info;          // < 0: this slot will get no more work; else rows | lazy layers to follow << 8 |
                     // value-only layers << 14 (0: keys, values and a query; 1 or 2: value rows of that many lazy
                     // layers in areas A, B) | raw logits wanted << 16
  long long glog;    // offset into p.logits of this chunk's first row
};
__device__ __forceinline__ int pack_info(int nrows, int nfol, int vonly, int want_logits) {
  return nrows | (nfol << 8) | (vonly << 14) | (want_logits << 16);
}

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

// The value pass of one consumer warp over its TR rows of a tile area: lane `lane` owns D/32 output dims and walks
// the rows; pr[g] is the probability of row g*8 + lane/4 (the same in the four lanes of a row's quad).  Rows past
// the warp's last one (nmine) carry probability 0 and re-read the last valid row: no branches.
template <typename T, int D, int TR>
__device__ __forceinline__ void value_pass(const unsigned char* warp_rows, int lane, int nmine, const float (&pr)[TR / 8],
                                           u64 (&acc2)[D / 64]) {
  constexpr int DPL = D / 32, ROWB = D * (int)sizeof(T);
#pragma unroll
  for (int i = 0; i < DPL / 2; ++i) acc2[i] = 0ull;
  const unsigned char* vrow = warp_rows + lane * (DPL * (int)sizeof(T));
#pragma unroll
  for (int rr = 0; rr < TR; ++rr) {
    const float pv = __shfl_sync(0xffffffffu, pr[rr / 8], (rr % 8) * 4);
    u64 v2[DPL / 2];
    load_pairs<T, DPL>(vrow + (size_t)min(rr, nmine - 1) * ROWB, v2);
    const u64 pp = pack2(pv, pv);
#pragma unroll
    for (int i = 0; i < DPL / 2; ++i) fma2(acc2[i], pp, v2[i]);
  }
}
// a lane's share of a warp's un-normalised result
template <int DPL>
__device__ __forceinline__ void store_acc(float* dst, const u64 (&acc2)[DPL / 2]) {
#pragma unroll
  for (int i = 0; i < DPL / 2; ++i) {
    float lo, hi;
    split2(acc2[i], lo, hi);
    *reinterpret_cast<float2*>(dst + 2 * i) = make_float2(lo, hi);
  }
}

// What the value-only uses that follow an item need to know of it (kept in shared memory per ring slot, not in
// the manager's registers).
struct Chain {
  const unsigned char* srcV;  // first value row of the chunk in the item's own layer
  int oidx, lb, l_rel, nrows, has_new, is_vis;
};

// A consumer warp's part of a value-only use (QK heredity): area A (and B when vonly == 2) of the slot holds
// the value rows of a lazy layer; the probabilities were left in `prob` by the item's own use (another group's
// warp with the same share of the rows).  The first layer's result goes to res0 (the group's result area), the
// second over the warp's own rows of area A.  Kept out of line: the plain path pays nothing for it.  Returns
// false when the wait for area B ran out.
template <typename T, int D, int TR>
__device__ __noinline__ bool consume_values(const unsigned char* areaA, const unsigned char* areaB, const float* prob,
                                            float* res0, uint64_t* barB, uint32_t parB, int vonly, int base, int nrows,
                                            int lane, volatile int* abort_flag, int* status) {
  constexpr int DPL = D / 32, ROWB = D * (int)sizeof(T), GR = TR / 8;
  const bool active = base < nrows;
  const int nmine = min(TR, nrows - base);
  float pr[GR];
  if (active) {
#pragma unroll
    for (int g = 0; g < GR; ++g) pr[g] = prob[base + g * 8 + (lane >> 2)];
    u64 acc2[DPL / 2];
    value_pass<T, D, TR>(areaA + (size_t)base * ROWB, lane, nmine, pr, acc2);
    store_acc<DPL>(res0 + lane * DPL, acc2);
    __syncwarp();  // every lane has read the warp's rows of area A before the next result goes there
  }
  if (vonly == 2) {
    if (!ring_wait(barB, parB, abort_flag, status)) return false;
    if (active) {
      u64 acc2[DPL / 2];
      value_pass<T, D, TR>(areaB + (size_t)base * ROWB, lane, nmine, pr, acc2);
      store_acc<DPL>(reinterpret_cast<float*>(const_cast<unsigned char*>(areaA) + (size_t)base * ROWB) + lane * DPL, acc2);
    }
  }
  return true;
}

// The manager's part of a value-only use: the value rows of the item's chunk (`c`) in lazy layers f0 .. f0+n-1
// (n = 1 or 2) go to tile areas A and B of the slot.  Out of line for the same reason.
template <typename T, int D>
__device__ __noinline__ void issue_values(const StepParams& p, const Chain* chain, ItemDesc* desc, unsigned char* areaA,
                                          unsigned char* areaB, uint64_t* barA, uint64_t* barB, int f0, int n, int lane,
                                          volatile int* abort_flag) {
  constexpr int ROWB = D * (int)sizeof(T), VPR = ROWB / 16, LN = VPR <= 16 ? VPR : 16, NV = VPR / LN;
  const Chain c = *chain;
  const int H = p.H;
  const size_t layer_bytes = (size_t)p.B * H * (size_t)p.lbh_stride * sizeof(T);  // one layer of cache blocks
  if (c.is_vis) {  // rows the previous step's selection may still be moving
    for (int j = 0; j < n; ++j)
      if (p.req[c.l_rel + f0 + j] &&
          !flag_wait(p.flags + c.lb + (f0 + j) * p.B, p.req[c.l_rel + f0 + j], abort_flag, p.status))
        return;
  }
  if (c.has_new) {  // the layers' newest value rows: lanes [0, LN) layer f0, [LN, 2 LN) the next one
    const int j = lane / LN;
    if (j < n) {
      const T* src = reinterpret_cast<const T*>(p.v_new) + (long long)(c.oidx + (f0 + j) * p.B * H) * D;
      unsigned char* dstg = const_cast<unsigned char*>(c.srcV) + (f0 + j) * layer_bytes + (size_t)(c.nrows - 1) * ROWB;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int cc = (lane % LN) + i * LN;
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(src) + cc);
        reinterpret_cast<uint4*>(dstg)[cc] = v;
        *reinterpret_cast<uint4*>((j ? areaB : areaA) + (size_t)(c.nrows - 1) * ROWB + cc * 16) = v;
      }
    }
    __syncwarp();
  }
  if (lane == 0) {
    desc->info = pack_info(c.nrows, 0, n, 0);
    const uint32_t kb = (uint32_t)(c.nrows - (c.has_new ? 1 : 0)) * ROWB;
    if (n == 2) {
      if (kb) {
        mbar_expect_tx(barB, kb);
        bulk_g2s(areaB, c.srcV + (f0 + 1) * layer_bytes, kb, barB);
      } else {
        mbar_arrive(barB);
      }
    }
    if (kb) {
      mbar_expect_tx(barA, kb);
      bulk_g2s(areaA, c.srcV + f0 * layer_bytes, kb, barA);
    } else {
      mbar_arrive(barA);
    }
  }
}

// FAT: the launch has items that carry lazy layers.  The host picks the plain instantiation when no layer of
// the call is lazy, so that path pays nothing (registers, code size) for the other.
template <typename T, int D, bool FAT>
__global__ void __launch_bounds__(kAttendThreads, 2) st3_attend_kernel(const __grid_constant__ StepParams p) {
  constexpr int EPL = 16 / sizeof(T);      // elements per 16-byte chunk
  constexpr int ROWB = D * sizeof(T);      // bytes per row
  constexpr int CPL = ROWB / 64;           // 16-byte chunks per lane (a lane owns a quarter row)
  constexpr int kTileBytes = ROWB >= 512 ? 32768 : 16384;  // K (and V) bytes of one ring slot
  constexpr int RMAX = kTileBytes / ROWB;  // rows per item: 64 (128 for 128-byte rows)
  constexpr int TR = RMAX / kGroupWarps;   // rows per consumer warp
  constexpr int GR = TR / 8;               // groups of 8 rows per warp
  constexpr int DPL = D / 32;              // output dims per lane when a warp holds one vector
  constexpr int SLOTB = 2 * kTileBytes + kQBytes;
  static_assert(4 * D <= TR * ROWB, "a warp's result vector must fit its own rows of a tile area");
  static_assert(CPL >= 2 && CPL <= 8 && GR >= 1, "unsupported row size");

  extern __shared__ __align__(128) unsigned char smem[];
  // one barrier set per (slot, consumer group): a group sees every phase of its own barriers, so
  // phase parity is never ambiguous
  // s_fullK / s_fullV: tile area A / B of the slot has landed; s_done: the group is done with the use.  Waiters
  // keep their own phase bit per barrier.
  __shared__ __align__(8) uint64_t s_fullK[kSlots][kGroups], s_fullV[kSlots][kGroups], s_done[kSlots][kGroups];
  __shared__ ItemDesc s_desc[kSlots];
  // what the value-only uses that follow an item need to know of it
  __shared__ Chain s_chain[FAT ? kSlots : 1];
  // the probabilities of the slot's last item with lazy layers (per row, relative to its warp's maximum)
  __shared__ float s_prob[FAT ? kSlots : 1][FAT ? RMAX : 1];
  // What a consumer group leaves of a use: per warp the (maximum, sum) of its rows and its un-normalised result,
  // in an area of the group's own, so that the slot can be refilled before the manager has read them (the
  // group's next use of the slot comes two uses later, after the manager has dealt with this one).
  __shared__ float s_stat[kSlots][kGroups][kGroupWarps][2];
  __shared__ __align__(16) float s_res[kSlots][kGroups][kGroupWarps][D];
  __shared__ int s_abort;

  // The finish launch that follows may be set up while this kernel runs (its blocks take the SMs this grid's
  // blocks leave and wait there for the whole grid: no launch latency between the two kernels).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
      bool valid, has_new, is_vis, want_logits, lazy;
      int nrows, wait_for, wait_for_k;
      int l_rel, nfol;   // relative layer; lazy layers riding on the item
      int slot;          // index of the item's partial: item * H + h
      int oidx, lb;      // (relative layer, sequence, head) and (layer, sequence) indices
      const unsigned char *srcK, *srcV;  // first key / value row of the chunk
      const T* srcQ;
      long long glog;  // offset into p.logits of this chunk's first row
      uint4 nv[NV];  // the newest row (key lanes and value lanes), fetched ahead of the slot becoming free
    };
    int wcur = 0;  // working layer of the previous visual item: this warp's items arrive in increasing order
    int lb_ready = -1;  // the (l, b) whose visual rows were last seen released by the previous finish launch
    // the first item of every manager is fixed (no round trip to the counter before the first copy);
    // the counter starts behind those and hands out the rest
    int x_next = (int)blockIdx.x * kSlots + s;

    // (layer, sequence, head) index of relative layer lr
    auto lbh_of = [&](int lr, int b, int h) { return ((long long)(p.layer_begin + lr) * p.B + b) * H + h; };
    auto oidx_of = [&](int lr, int b, int h) { return ((long long)lr * p.B + b) * H + h; };
    // first key (kv = 0) or value (kv = 1) row of the region an item of relative layer lr reads
    auto region_of = [&](int lr, int b, int h, bool is_vis, int kv) {
      T* blk = reinterpret_cast<T*>(p.cache) + lbh_of(lr, b, h) * p.lbh_stride;
      if (is_vis) return blk + (long long)kv * p.Nv * D;
      return blk + 2LL * p.Nv * D + (long long)kv * p.cap_txt * D;
    };

    auto decode = [&](Dec& d) {
      const int x = __shfl_sync(0xffffffffu, x_next, 0);
      d.valid = (unsigned)x < (unsigned)total;
      if (!d.valid) return;
      if (lane == 0)  // prefetch the index after this one
        x_next = p.first_dynamic + (int)(atomicAdd(reinterpret_cast<unsigned*>(p.work_counter), 1u) - p.counter_base);
      // Order of work: the text (and system) chunks of every layer first, then the visual chunks layer by
      // layer.  Only visual rows are moved by the previous step's finish launch, which is still running when
      // this launch starts: what does not depend on it comes first (+4 % tokens/s at B=1 over a layer-major
      // order, whose visual chunks of the first pruning layers waited ~4 us each for their flag).  A partial's
      // slot keeps the layer-major numbering (visual chunks, then text chunks of each (l, b)) that the finish
      // kernel reads.
      const int xi = (int)fast_div((unsigned)x, p.h_mul, p.h_shift);
      const int h = x - xi * H;
      const bool is_vis = xi >= p.text_items;
      int l_rel, b, c, cv;
      if (!is_vis) {
        const int w = (int)fast_div((unsigned)xi, p.bct_mul, p.bct_shift);
        l_rel = p.wlayer[w];
        const int rem = xi - w * p.B * p.ct;
        b = (int)fast_div((unsigned)rem, p.ct_mul, p.ct_shift);
        cv = p.cvp[l_rel + 1] - p.cvp[l_rel];
        c = cv + rem - b * p.ct;
      } else {
        const int iv = xi - p.text_items;
        while (wcur + 1 < p.nwork && iv >= p.B * p.wcvp[wcur + 1]) ++wcur;
        l_rel = p.wlayer[wcur];
        cv = p.cvp[l_rel + 1] - p.cvp[l_rel];
        const int off = iv - p.B * p.wcvp[wcur];
        b = (int)fast_div((unsigned)off, p.cv_mul[l_rel], p.cv_shift[l_rel]);
        c = off - b * cv;
      }
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
      d.is_vis = is_vis; d.l_rel = l_rel;
      d.slot = (p.lstart[l_rel] + b * (cv + p.ct) + c) * H + h;  // partials are numbered layer-major
      d.oidx = (l_rel * p.B + b) * H + h;
      d.nfol = FAT ? p.nfol[l_rel] : 0;
      d.want_logits = is_vis && p.ntgt[l_rel] < p.ncur[l_rel] && p.src_layer[l_rel] == p.layer_begin + l_rel;
      const int lb = (p.layer_begin + l_rel) * p.B + b;
      d.lb = lb;
      d.wait_for = is_vis && lb != lb_ready ? p.req[l_rel] : 0;
      if (d.wait_for && ld_acquire(p.flags + lb) - d.wait_for >= 0) {  // looked up here, off the critical path
        d.wait_for = 0;
        lb_ready = lb;
      }
      // QK heredity (Eq. 6): a lazy layer with items of its own attends with the query and the keys of its
      // source layer and its own values; the two layers hold the same tokens in the same order
      const int ls = p.lazy_src[l_rel];
      const int lk = ls < 0 ? l_rel : ls;  // whose keys and query
      d.lazy = ls >= 0;
      d.wait_for_k = is_vis && ls >= 0 ? p.req[ls] : 0;  // the source's rows as well
      d.srcK = reinterpret_cast<const unsigned char*>(region_of(lk, b, h, is_vis, 0)) + (size_t)r0 * ROWB;
      d.srcV = reinterpret_cast<const unsigned char*>(region_of(l_rel, b, h, is_vis, 1)) + (size_t)r0 * ROWB;
      d.srcQ = reinterpret_cast<const T*>(p.q) + oidx_of(lk, b, h) * D;
      d.glog = lbh_of(l_rel, b, h) * p.Nv + r0;
      if (d.has_new && lane < 2 * LN) {
        // newest row: fetched from the step's inputs now, stored when the slot is free
        const T* src = lane / LN ? reinterpret_cast<const T*>(p.v_new) + oidx_of(l_rel, b, h) * D
                                 : reinterpret_cast<const T*>(p.k_new) + oidx_of(ls < 0 ? l_rel : ls, b, h) * D;
#pragma unroll
        for (int i = 0; i < NV; ++i) d.nv[i] = __ldg(reinterpret_cast<const uint4*>(src) + (lane % LN) + i * LN);
      }
    };
    // Starts the copies of a decoded item into this (free) slot.
    auto issue = [&](const Dec& d, int g) {  // g: the consumer group this use of the slot belongs to
      if (d.wait_for) {
        if (!flag_wait(p.flags + d.lb, d.wait_for, abort_flag, p.status)) return;
        lb_ready = d.lb;
      }
      if (d.wait_for_k &&  // the source layer's (l, b): the same sequence, lazy_src layers lower
          !flag_wait(p.flags + d.lb + (p.lazy_src[d.l_rel] - d.l_rel) * p.B, d.wait_for_k, abort_flag, p.status))
        return;
      if (d.has_new) {
        if (lane < 2 * LN) {
          const int kv = lane / LN;
          // the row's place in the cache is the chunk's last row; a lazy layer stores no key: its source does
          unsigned char* dstg = const_cast<unsigned char*>(kv ? d.srcV : d.srcK) + (size_t)(d.nrows - 1) * ROWB;
          if (!kv && d.lazy) dstg = nullptr;
#pragma unroll
          for (int i = 0; i < NV; ++i) {
            const int cc = (lane % LN) + i * LN;
            if (dstg) reinterpret_cast<uint4*>(dstg)[cc] = d.nv[i];
            *reinterpret_cast<uint4*>((kv ? sV : sK) + (size_t)(d.nrows - 1) * ROWB + cc * 16) = d.nv[i];
          }
        }
        __syncwarp();
      }
      if (lane == 0) {
        if constexpr (FAT) {
          if (d.nfol > 0) {
            Chain& c = s_chain[s];
            c.srcV = d.srcV; c.oidx = d.oidx; c.lb = d.lb; c.l_rel = d.l_rel; c.nrows = d.nrows;
            c.has_new = d.has_new; c.is_vis = d.is_vis;
          }
        }
        ItemDesc& sd = s_desc[s];
        sd.info = pack_info(d.nrows, d.nfol, 0, d.want_logits);
        sd.glog = d.glog;
        const uint32_t kb = (uint32_t)(d.nrows - (d.has_new ? 1 : 0)) * ROWB;
        mbar_expect_tx(&s_fullK[s][g], kb + ROWB);  // K rows + the query (D elements = ROWB bytes)
        bulk_g2s(sQ, d.srcQ, ROWB, &s_fullK[s][g]);
        if (kb) {
          bulk_g2s(sK, d.srcK, kb, &s_fullK[s][g]);
          mbar_expect_tx(&s_fullV[s][g], kb);
          bulk_g2s(sV, d.srcV, kb, &s_fullV[s][g]);
        } else {
          mbar_arrive(&s_fullV[s][g]);
        }
      }
    };
    Dec nxt;
    decode(nxt);
    // Use u of this slot belongs to consumer group (u + s) % kGroups.
    if (nxt.valid) issue(nxt, s % kGroups);
    // the item in the slot: what is still needed of it once its copies are on their way
    bool cur_valid = nxt.valid;
    int cur_nrows = nxt.nrows, cur_slot = nxt.slot, cur_nfol = nxt.nfol, cur_lrel = nxt.l_rel;
    unsigned ph_done = 0;  // phase bits of the two groups' s_done barriers
    bool have_nxt = false;
    int f0 = 0, fn = 1;    // the layers of the item this use works on: f0 .. f0+fn-1 layers above the item's own
    float M = -INFINITY, Lsum = 0.f, wgt = 0.f;  // of the item: maximum, sum, this lane's warp's weight
    int nw = 0;
    for (int use = 0; cur_valid; ++use) {
      if (!have_nxt) { decode(nxt); have_nxt = true; }  // in the shadow of this item's copies and the consumers' work
      const int g = (use + s) % kGroups;
      // what follows this use: more lazy layers of the same item, or the next item
      const int fnext = f0 + fn;
      const int nn = FAT ? min(2, cur_nfol - fnext + 1) : 0;   // > 0: a value-only use for layers fnext ..
      // ---- wait for this use's consumer group ----
      if (!ring_wait(&s_done[s][g], (ph_done >> g) & 1u, abort_flag, p.status)) break;
      ph_done ^= 1u << g;
      // the partial slots of this use's layers: same chunk of the same rows, f layers up
      const int slot0 = cur_slot + (FAT ? (p.lstart[cur_lrel + f0] - p.lstart[cur_lrel]) * H : 0);
      auto publish = [&](int slot, const float (&v)[DPL]) {  // plain stores: the next kernel merges the partials
        float* dst = p.part_acc + (long long)slot * D + lane * DPL;
        if constexpr (DPL == 4) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[DPL - 2], v[DPL - 1]);
        else *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
        if (lane == 0) *reinterpret_cast<float2*>(p.part_ml + 2 * (long long)slot) = make_float2(M, Lsum);
      };
      float po[DPL];
      if constexpr (FAT) {
        if (fn == 2) {
          // the second layer of a value-only use lies over each warp's own rows of area A: read before the refill
#pragma unroll
          for (int j = 0; j < DPL; ++j) po[j] = 0.f;
#pragma unroll
          for (int w = 0; w < kGroupWarps; ++w) {
            const float ww = __shfl_sync(0xffffffffu, wgt, w);
            if (w < nw) {
              const float* res = reinterpret_cast<const float*>(sK + (size_t)w * TR * ROWB) + lane * DPL;
#pragma unroll
              for (int j = 0; j < DPL; j += 2) {
                const float2 v2 = *reinterpret_cast<const float2*>(res + j);
                po[j] = fmaf(v2.x, ww, po[j]); po[j + 1] = fmaf(v2.y, ww, po[j + 1]);
              }
            }
          }
          __syncwarp();  // every lane is done reading the slot before it is refilled
          publish(cur_slot + (p.lstart[cur_lrel + f0 + 1] - p.lstart[cur_lrel]) * H, po);
        }
      }
      // ---- refill the slot at once: what the group left lies outside the tile areas ----
      const bool own_use = f0 == 0;  // the item's own use (keys, values, query): it produced the statistics
      const int nrows_use = cur_nrows;
      if (nn > 0) {
        if constexpr (FAT) {
          const int gn = (use + 1 + s) % kGroups;
          __syncwarp();
          issue_values<T, D>(p, &s_chain[s], &s_desc[s], sK, sV, &s_fullK[s][gn], &s_fullV[s][gn], fnext, nn, lane,
                             abort_flag);
        }
        f0 = fnext; fn = nn;
      } else {
        if (nxt.valid) issue(nxt, (use + 1 + s) % kGroups);
        cur_valid = nxt.valid;
        cur_nrows = nxt.nrows; cur_slot = nxt.slot; cur_nfol = nxt.nfol; cur_lrel = nxt.l_rel;
        have_nxt = false;
        f0 = 0; fn = 1;
      }
      // ---- fold the warps' results (each relative to its warp's own maximum) and publish the partial ----
      if (own_use) {
        nw = (nrows_use + TR - 1) / TR;
        const float mw = lane < nw ? s_stat[s][g][lane][0] : -INFINITY;
        const float lw = lane < nw ? s_stat[s][g][lane][1] : 0.f;
        M = warp_max(mw);
        wgt = lane < nw ? fast_exp2(mw - M) : 0.f;
        Lsum = warp_sum(lw * wgt);
      }
#pragma unroll
      for (int j = 0; j < DPL; ++j) po[j] = 0.f;
#pragma unroll
      for (int w = 0; w < kGroupWarps; ++w) {
        const float ww = __shfl_sync(0xffffffffu, wgt, w);
        if (w < nw) {
          const float* res = &s_res[s][g][w][lane * DPL];
#pragma unroll
          for (int j = 0; j < DPL; j += 2) {
            const float2 v2 = *reinterpret_cast<const float2*>(res + j);
            po[j] = fmaf(v2.x, ww, po[j]); po[j + 1] = fmaf(v2.y, ww, po[j + 1]);
          }
        }
      }
      publish(slot0, po);
    }
    // out of work (or aborted): an end marker for each consumer group, on the group's own barrier
    if (lane == 0) {
      s_desc[s].info = -1;
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
    unsigned phf = 0;  // this warp's phase bits: bit 2s for tile area A of slot s, bit 2s+1 for area B
    for (int round = 0; live; ++round) {
      const int s = round % kSlots;
      const int use = round / kSlots;  // round r is use r / kSlots of slot r % kSlots
      if ((use + s) % kGroups != grp || !(live & (1u << s))) continue;
      const unsigned bitA = 1u << (2 * s), bitB = 2u << (2 * s);
      if (!ring_wait(&s_fullK[s][grp], (phf & bitA) ? 1u : 0u, abort_flag, p.status)) break;
      phf ^= bitA;
      const int info = s_desc[s].info;
      const int nrows = info < 0 ? -1 : info & 0xff;
      if (nrows < 0) { live &= ~(1u << s); continue; }
      const int nfol = FAT ? (info >> 8) & 0x3f : 0;
      const int vonly = FAT ? (info >> 14) & 3 : 0;
      const int base = w * TR;
      const bool active = base < nrows;  // a warp without rows still follows the use's barriers
      unsigned char* sK = smem + (size_t)s * SLOTB;
      unsigned char* sV = sK + kTileBytes;
      float pr[GR], m = -INFINITY, lsum = 0.f;
      // ---- V pass: a lane owns DPL output dims and walks this warp's rows ----
      const int nmine = min(TR, nrows - base);
      auto vpass = [&](const unsigned char* area, u64 (&acc2)[DPL / 2]) {
        value_pass<T, D, TR>(area + (size_t)base * ROWB, lane, nmine, pr, acc2);
      };
      // a warp's un-normalised result, a [D] vector, goes to the group's own result area; the second layer of a
      // value-only use goes over the warp's own (consumed) rows of area A
      auto store_result = [&](int f, const u64 (&acc2)[DPL / 2]) {
        store_acc<DPL>((f == 0 ? &s_res[s][grp][w][0] : reinterpret_cast<float*>(sK + (size_t)base * ROWB)) + lane * DPL,
                       acc2);
      };
      if constexpr (FAT) {
        if (vonly > 0) {  // value-only use: a lazy layer's value rows and the probabilities the item left
          const bool okv = consume_values<T, D, TR>(sK, sV, s_prob[s], &s_res[s][grp][w][0], &s_fullV[s][grp],
                                                    (phf & bitB) ? 1u : 0u, vonly, base, nrows, lane, abort_flag,
                                                    p.status);
          if (!okv) break;
          if (vonly == 2) phf ^= bitB;
          __syncwarp();
          if (lane == 0) mbar_arrive(&s_done[s][grp]);
          continue;
        }
      }
      if (active) {
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
        m = sl[0];
#pragma unroll
        for (int g = 1; g < GR; ++g) m = fmaxf(m, sl[g]);
        m = warp_max(m);
        if ((info >> 16 & 1) && c4 == 0) {
          float* glog = p.logits + s_desc[s].glog;
#pragma unroll
          for (int g = 0; g < GR; ++g)
            if (ok[g]) glog[base + g * 8 + r8] = sl[g];
        }
#pragma unroll
        for (int g = 0; g < GR; ++g) {
          pr[g] = ok[g] ? fast_exp2(sl[g] - m) : 0.f;
          if (c4 == 0) lsum += pr[g];
        }
        lsum = warp_sum(lsum);
        if constexpr (FAT) {
          if (nfol > 0 && c4 == 0) {  // lazy layers follow: they will need these (0 for rows past the end)
#pragma unroll
            for (int g = 0; g < GR; ++g) s_prob[s][base + g * 8 + r8] = pr[g];
          }
        }
      }
      if (!ring_wait(&s_fullV[s][grp], (phf & bitB) ? 1u : 0u, abort_flag, p.status)) break;
      phf ^= bitB;
      if (active) {
        u64 acc2[DPL / 2];
        vpass(sV, acc2);
        store_result(0, acc2);
        if (lane == 0) { s_stat[s][grp][w][0] = m; s_stat[s][grp][w][1] = lsum; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_done[s][grp]);
    }
  }
  // This grid started without waiting for the launch before it (flags order what they share).  It must not
  // *complete* before that launch has, though: the finish launch after this one waits for this grid only.
  asm volatile("griddepcontrol.wait;" ::: "memory");
}


}  // namespace

#endif  // ST3_ATTEND_CUH_
