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
      bool valid, has_new;
      int nrows, nbulk, want_logits, wait_for, wait_for_k;
      long long slot, lbh, oidx, oidx_q, glog, lb, lb_k;
      const unsigned char *srcK, *srcV;
      T *newK, *newV;
      uint4 nv[NV];
    };
    int lcur = 0;  // layer of the previous visual item: this warp's items arrive in increasing order
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
        l_rel = (int)fast_div((unsigned)xi, p.bct_mul, p.bct_shift);
        const int rem = xi - l_rel * p.B * p.ct;
        b = (int)fast_div((unsigned)rem, p.ct_mul, p.ct_shift);
        cv = p.cvp[l_rel + 1] - p.cvp[l_rel];
        c = cv + rem - b * p.ct;
      } else {
        const int iv = xi - p.text_items;
        while (lcur + 1 < p.layer_count && iv >= p.B * p.cvp[lcur + 1]) ++lcur;
        l_rel = lcur;
        cv = p.cvp[l_rel + 1] - p.cvp[l_rel];
        const int off = iv - p.B * p.cvp[l_rel];
        b = (int)fast_div((unsigned)off, p.cv_mul[l_rel], p.cv_shift[l_rel]);
        c = off - b * cv;
      }
      const int l = p.layer_begin + l_rel;
      const int item = p.lstart[l_rel] + b * (cv + p.ct) + c;
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
  // This grid started without waiting for the launch before it (flags order what they share).  It must not
  // *complete* before that launch has, though: the finish launch after this one waits for this grid only.
  asm volatile("griddepcontrol.wait;" ::: "memory");
}


}  // namespace

#endif  // ST3_ATTEND_CUH_
