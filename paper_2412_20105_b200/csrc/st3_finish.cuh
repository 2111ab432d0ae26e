// Part of the ST^3 library for sm_100a; included by st3.cu only.
#ifndef ST3_FINISH_CUH_
#define ST3_FINISH_CUH_
#include "st3_common.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// Merge partials, visual scores, top-k (Eq. 3), in-place compaction (Eq. 7's eviction)
// ------------------------------------------------------------------------------------------
// Two blocks per (layer, sequence), on different SMs, that never wait for each other:
//   OUT block   merges the chunk partials of every head into the attention output (a warp per head);
//   TRIM block  merges only the (max, sum) pairs, turns the raw logits into head-summed
//               probabilities, radix-selects the rows to keep, pairs holes with kept tail rows and
//               moves the rows.
// Both are chains of dependent memory round trips, so every phase issues all its loads first.
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

// NT threads per block: 1024, or 512 (two blocks per SM) when a launch has more (layer, sequence) units than the GPU
// can hold blocks: the work of a unit is a chain of memory round trips, and more units in flight end sooner.
template <typename T, int D, int NT>
__global__ void __launch_bounds__(NT, 1024 / NT) st3_finish_kernel(const StepParams p) {
  constexpr int kFinishThreads = NT, kFinishWarps = NT / 32;
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

  // This launch may have been set up while the attention launch before it was still running: wait for that
  // whole grid (and, through it, for everything earlier in the stream).  Then the next step's attention launch
  // may start; it waits on p.flags for what this launch changes.
  asm volatile("griddepcontrol.wait;" ::: "memory");
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


}  // namespace

#endif  // ST3_FINISH_CUH_
