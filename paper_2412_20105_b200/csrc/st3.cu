// ST^3 decode-step attention over a trimmed visual KV cache: sm_100a kernels and the C ABI.
//
// Cache layout (device, caller's workspace).  For every (layer l, sequence b, head h) one block
//   [ K_vis : Nv x D ][ V_vis : Nv x D ][ K_txt : cap x D ][ V_txt : cap x D ]
// with cap = sys_len + max_text_len + max_decode_steps.  The visual rows live in their own
// region so that evicting them never shifts system / text / generated rows; the text region
// holds [S | I | O_1.. ] in order.  ids[l][b][i] is the ORIGINAL visual index of visual row i.
//
// One step = two launches (kernels in st3_attend.cuh and st3_finish.cuh, shared pieces in st3_common.cuh):
//   st3_attend_kernel   persistent, warp-specialised blocks stream (layer, sequence, head, row chunk)
//                       work items through a shared-memory ring with bulk asynchronous copies and
//                       leave one softmax partial (m, l, acc) per item, plus the raw logits of visual
//                       rows for layers that evict at this step; the newest token's row is appended
//                       on the way.
//   st3_finish_kernel   per (layer, sequence) one block merges the partials of every head into the
//                       attention output and one block scores the visual rows, radix-selects the rows
//                       to keep (ties toward the lower original index) and fills the holes among the
//                       first n_new rows with the kept rows of the tail.
// A step's finish launch overlaps the next step's attention launch (programmatic dependent launch,
// ordered by per-(layer, sequence) flags).  The work decomposition is computed on the host from the
// schedule (row counts are a pure function of layer and step), so no table is uploaded per step.
// This file holds the host logic and the C ABI.
#include "st3.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <new>
#include <vector>

#include "st3_common.cuh"
#include "st3_attend.cuh"
#include "st3_finish.cuh"

namespace {

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
  size_t elem, cache, part_ml, part_acc, part_ml_bytes, part_acc_bytes, logits, logits_bytes, head_stat, mass, ids, n_cur, flags, text_len, status,
      io_bytes,       // one of q / k_new / v_new / out over all layers
      stage_in,       // two slots of [q | k_new | v_new] for the host-buffer decode step
      stage_o,        // two slots of out
      stage_pq,       // q_last and out of the host-buffer prefill
      stage_po,
      prompt_bytes,   // K (or V) rows of one layer's prompt
      stage_prompt,   // two slots of [K | V] of one layer (only with host_prefill)
      total;
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
  L.io_bytes = align_up(lbh * c->head_dim * L.elem, 256);
  L.stage_in = take(2 * 3 * L.io_bytes);
  L.stage_o = take(2 * L.io_bytes);
  L.stage_pq = take(L.io_bytes);
  L.stage_po = take(L.io_bytes);
  L.prompt_bytes = align_up((size_t)c->batch * c->num_heads * ((size_t)c->sys_len + c->num_visual + c->max_text_len) *
                                c->head_dim * L.elem, 256);
  L.stage_prompt = c->host_prefill ? take(2 * 2 * L.prompt_bytes) : off;
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
  bool overlap;                // st3_set_overlap: the attention launch may start before the launch ahead of it ends
  bool failed;                 // a launch failed half-way: host bookkeeping and device state may disagree
  // host-buffer calls: copies to the device and back travel on two streams of the library's own
  cudaStream_t s_h2d, s_d2h;
  cudaEvent_t ev_in[2], ev_k[2], ev_out[2];   // per decode staging slot: inputs landed / kernels done / out copied back
  cudaEvent_t ev_pin[2], ev_pk[2], ev_pq;     // per prompt staging slot: K/V landed / layer done; q_last staging free
  bool rec_k[2], rec_out[2], rec_pk[2], rec_pq;
  uint64_t hseq, pseq;                        // host-buffer decode steps / prompt layers so far (slot = low bit)
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
    st3_finish_kernel<T, D, kFinishThreads><<<(unsigned)(2 * p.layer_count * c.batch), kFinishThreads, ctx->finish_smem, st>>>(
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
    // With st3_set_overlap(ctx, 1) this is a programmatic dependent launch: it may start while the previous
    // step's finish launch is still running (that kernel allows it at its start); p.flags orders what the two
    // share.  The kernel reads the step's inputs without waiting for the launch ahead of it, which is only
    // right when those inputs were complete before that launch began - hence off unless the caller says so.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.first_dynamic / kSlots));
    cfg.blockDim = dim3(kAttendThreads);
    cfg.dynamicSmemBytes = (size_t)ctx->attend_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (!ctx->overlap || ctx->profiling || ingest || ctx->serialize_next) ? 0 : 1;
    bool fat = false;  // some item carries lazy layers (QK heredity): the instantiation that streams their values
    for (int i = 0; i < p.layer_count; ++i) fat = fat || p.nfol[i] != 0;
    if ((fat ? cudaLaunchKernelEx(&cfg, st3_attend_kernel<T, D, true>, p)
             : cudaLaunchKernelEx(&cfg, st3_attend_kernel<T, D, false>, p)) != cudaSuccess)
      return ST3_ERR_CUDA;
  }
  if (e1) cudaEventRecord(e1, st);
  {
    // Also a programmatic dependent launch: the attention kernel allows it at its start, the blocks become
    // resident as that grid drains and their first instruction waits for all of it.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * p.layer_count * c.batch));
    // half-size blocks, two per SM, once the units outnumber the blocks the GPU holds (see st3_finish.cuh)
    const bool half = 2 * p.layer_count * c.batch > 2 * ctx->num_sms && 2 * ctx->finish_smem <= 200 * 1024;
    cfg.blockDim = dim3(half ? kFinishThreads / 2 : kFinishThreads);
    cfg.dynamicSmemBytes = (size_t)ctx->finish_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->profiling ? 0 : 1;
    if ((half ? cudaLaunchKernelEx(&cfg, st3_finish_kernel<T, D, kFinishThreads / 2>, p)
              : cudaLaunchKernelEx(&cfg, st3_finish_kernel<T, D, kFinishThreads>, p)) != cudaSuccess)
      return ST3_ERR_CUDA;
  }
  if (e2) cudaEventRecord(e2, st);
  ctx->launches += 2;
  return cudaGetLastError() == cudaSuccess ? ST3_OK : ST3_ERR_CUDA;
}

template <typename T, int D>
st3_status set_attrs_t(st3_ctx* ctx) {
  if (cudaFuncSetAttribute(st3_attend_kernel<T, D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           ctx->attend_smem) != cudaSuccess ||
      cudaFuncSetAttribute(st3_attend_kernel<T, D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           ctx->attend_smem) != cudaSuccess)
    return ST3_ERR_CUDA;
  if (cudaFuncSetAttribute(st3_finish_kernel<T, D, kFinishThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           ctx->finish_smem) != cudaSuccess ||
      cudaFuncSetAttribute(st3_finish_kernel<T, D, kFinishThreads / 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
    make_fast_div((unsigned)(cv > 0 ? cv : 1), &p.cv_mul[i], &p.cv_shift[i]);
  }
  p.lstart[layer_count] = c.batch * (p.cvp[layer_count] + layer_count * p.ct);
  // Working layers: every layer except the lazy ones that ride on the items of the layer they inherit from
  // (their value rows follow the item through its ring slot, see st3_attend.cuh; a run of more than kMaxFollow
  // lazy layers would start a new group that reads the keys again).
  bool works[kMaxLayers];
  for (int i = 0, head = -1; i < layer_count; ++i) {
    const int s = p.lazy_src[i];
    const bool rides = s >= 0 && head >= 0 && (head == s || p.lazy_src[head] == s) &&
                       head + p.nfol[head] + 1 == i && p.nfol[head] < kMaxFollow &&
                       p.ncur[i] == p.ncur[head] && p.nold[i] == p.nold[head];
    works[i] = !rides;
    if (rides) p.nfol[head]++;
    else head = i;
  }
  // Order of the working layers inside the launch: those whose items are followed by lazy layers first.  Such an
  // item keeps its ring slot for several uses in a row; at the end of a launch, where little other work is left
  // to hide it, that chain would set the length of the tail.
  p.nwork = 0;
  p.wcvp[0] = 0;
  for (int pass = 0; pass < 2; ++pass)
    for (int i = 0; i < layer_count; ++i) {
      if (!works[i] || (p.nfol[i] != 0) != (pass == 0)) continue;
      p.wlayer[p.nwork] = (unsigned char)i;
      p.wcvp[p.nwork + 1] = p.wcvp[p.nwork] + (p.cvp[i + 1] - p.cvp[i]);
      p.nwork++;
    }
  make_fast_div((unsigned)c.num_heads, &p.h_mul, &p.h_shift);
  p.text_items = p.nwork * c.batch * p.ct;
  make_fast_div((unsigned)(c.batch * p.ct), &p.bct_mul, &p.bct_shift);
  make_fast_div((unsigned)p.ct, &p.ct_mul, &p.ct_shift);
  const long long total_items = (long long)c.batch * (p.cvp[layer_count] + (long long)layer_count * p.ct);
  const long long work_items = (long long)c.batch * (p.wcvp[p.nwork] + (long long)p.nwork * p.ct);
  if (total_items > L.max_items || work_items * c.num_heads > 0x3fffffffLL) return ST3_ERR_CAPACITY;
  p.total_work = (int)(work_items * c.num_heads);
  // blocks of the attention grid: as many as fit the GPU, fewer when the launch has fewer items than ring slots
  {
    const int full = ctx->num_sms * ctx->attend_ctas_per_sm, need = ceil_div(p.total_work, kSlots);
    p.first_dynamic = (need < full ? (need > 0 ? need : 1) : full) * kSlots;
  }

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
  if (s != ST3_OK) {
    // Some kernel of the call may already be enqueued (the device work counter, the flags and the cache then
    // move on without the host's bookkeeping): nothing later on this context can be trusted.
    ctx->failed = true;
    return s;
  }
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
  ctx->overlap = false;
  ctx->failed = false;
  ctx->profiling = false;
  ctx->ev_used = 0;
  ctx->s_h2d = ctx->s_d2h = nullptr;
  ctx->ev_pq = nullptr;
  for (int i = 0; i < 2; ++i) {
    ctx->ev_in[i] = ctx->ev_k[i] = ctx->ev_out[i] = ctx->ev_pin[i] = ctx->ev_pk[i] = nullptr;
    ctx->rec_k[i] = ctx->rec_out[i] = ctx->rec_pk[i] = false;
  }
  ctx->rec_pq = false;
  ctx->hseq = ctx->pseq = 0;
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
    if (cudaMemsetAsync(ctx->ws + L.mass, 0, L.stage_in - L.mass, nullptr) != cudaSuccess ||
        cudaStreamSynchronize(nullptr) != cudaSuccess)
      s = ST3_ERR_CUDA;
  }
  if (s == ST3_OK) {
    bool ok = cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->ev_pq, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->ev_k[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->ev_pin[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->ev_pk[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) s = ST3_ERR_CUDA;
  }
  if (s != ST3_OK) { st3_destroy(ctx); return s; }
  *out = ctx;
  return ST3_OK;
}

static st3_status prefill_common(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last,
                                 const void* k, const void* v, const int32_t* text_len, const float* scores,
                                 void* out, void* cuda_stream) {
  if (!ctx || !text_len) return ST3_ERR_INVALID_ARG;
  if (ctx->failed) return ST3_ERR_BAD_STATE;
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
  // A call that starts at layer 0, or that brings other text lengths, opens a new generation: every layer
  // must be prefilled again before it can decode.
  bool differs = !ctx->have_text;
  for (int b = 0; b < c.batch && !differs; ++b) differs = ctx->text_len[b] != text_len[b];
  if (differs || layer_begin == 0)
    for (int l = 0; l < c.num_layers; ++l) { ctx->last_step[l] = -1; ctx->logit_step[l] = -1; }
  if (differs) {
    for (int b = 0; b < c.batch; ++b) ctx->text_len[b] = text_len[b];
    ctx->max_text = mx;
    ctx->have_text = true;
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
  if (ctx->failed) return ST3_ERR_BAD_STATE;
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
  if (ctx->failed) return ST3_ERR_BAD_STATE;
  const st3_config& c = ctx->cfg;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c.num_layers) return ST3_ERR_INVALID_ARG;
  const Layout& L = ctx->lay;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)layer_count * c.batch * c.num_heads * c.head_dim * L.elem;
  const int slot = (int)(ctx->hseq & 1);
  unsigned char* dq = ctx->ws + L.stage_in + (size_t)slot * 3 * L.io_bytes;
  unsigned char* dk = dq + bytes;
  unsigned char* dv = dk + bytes;
  unsigned char* dout = ctx->ws + L.stage_o + (size_t)slot * L.io_bytes;
  const unsigned char* hq = static_cast<const unsigned char*>(q_host);
  const unsigned char* hk = static_cast<const unsigned char*>(k_new_host);
  const unsigned char* hv = static_cast<const unsigned char*>(v_new_host);
  // inputs: on the copy-in stream, once the kernels that last read this staging slot (two steps ago) are done
  if (ctx->rec_k[slot] && cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_k[slot], 0) != cudaSuccess) return ST3_ERR_CUDA;
  if (hk == hq + bytes && hv == hk + bytes) {
    // q, k_new, v_new packed back to back by the caller: one copy instead of three
    if (cudaMemcpyAsync(dq, hq, 3 * bytes, cudaMemcpyHostToDevice, ctx->s_h2d) != cudaSuccess) return ST3_ERR_CUDA;
  } else if (cudaMemcpyAsync(dq, hq, bytes, cudaMemcpyHostToDevice, ctx->s_h2d) != cudaSuccess ||
             cudaMemcpyAsync(dk, hk, bytes, cudaMemcpyHostToDevice, ctx->s_h2d) != cudaSuccess ||
             cudaMemcpyAsync(dv, hv, bytes, cudaMemcpyHostToDevice, ctx->s_h2d) != cudaSuccess) {
    return ST3_ERR_CUDA;
  }
  if (cudaEventRecord(ctx->ev_in[slot], ctx->s_h2d) != cudaSuccess ||
      cudaStreamWaitEvent(st, ctx->ev_in[slot], 0) != cudaSuccess)
    return ST3_ERR_CUDA;
  // the slot's output staging must have been copied back (two steps ago) before the kernels write it again
  if (ctx->rec_out[slot] && cudaStreamWaitEvent(st, ctx->ev_out[slot], 0) != cudaSuccess) return ST3_ERR_CUDA;
  const st3_status s = st3_decode_step(ctx, step, layer_begin, layer_count, dq, dk, dv, dout, cuda_stream);
  if (s != ST3_OK) return s;
  if (cudaEventRecord(ctx->ev_k[slot], st) != cudaSuccess) return ST3_ERR_CUDA;
  ctx->rec_k[slot] = true;
  // output: on the copy-out stream, behind the kernels
  if (cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_k[slot], 0) != cudaSuccess ||
      cudaMemcpyAsync(out_host, dout, bytes, cudaMemcpyDeviceToHost, ctx->s_d2h) != cudaSuccess ||
      cudaEventRecord(ctx->ev_out[slot], ctx->s_d2h) != cudaSuccess)
    return ST3_ERR_CUDA;
  ctx->rec_out[slot] = true;
  ctx->hseq++;
  return ST3_OK;
}

st3_status st3_prefill_select_host(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last_host,
                                   const void* k_host, const void* v_host, const int32_t* text_len, void* out_host,
                                   void* cuda_stream) {
  if (!ctx || !q_last_host || !k_host || !v_host || !out_host || !text_len) return ST3_ERR_INVALID_ARG;
  if (ctx->failed || !ctx->cfg.host_prefill) return ST3_ERR_BAD_STATE;
  const st3_config& c = ctx->cfg;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c.num_layers) return ST3_ERR_INVALID_ARG;
  if (c.lazy_mask) return ST3_ERR_UNSUPPORTED;
  const Layout& L = ctx->lay;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t lq = (size_t)c.batch * c.num_heads * c.head_dim * L.elem;  // one layer of q_last / out
  const size_t lp = (size_t)c.batch * c.num_heads * ((size_t)c.sys_len + c.num_visual + c.max_text_len) * c.head_dim * L.elem;
  unsigned char* dq = ctx->ws + L.stage_pq;
  unsigned char* dout = ctx->ws + L.stage_po;
  // q_last of every layer in one copy, once the kernels of an earlier call are done with the staging area
  if (ctx->rec_pq && cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_pq, 0) != cudaSuccess) return ST3_ERR_CUDA;
  if (cudaMemcpyAsync(dq, q_last_host, lq * layer_count, cudaMemcpyHostToDevice, ctx->s_h2d) != cudaSuccess)
    return ST3_ERR_CUDA;
  for (int i = 0; i < layer_count; ++i) {
    const int slot = (int)(ctx->pseq & 1);
    unsigned char* dk = ctx->ws + L.stage_prompt + (size_t)slot * 2 * L.prompt_bytes;
    unsigned char* dv = dk + L.prompt_bytes;
    // layer i's rows move while the layer before it is ingested, attended and trimmed
    if (ctx->rec_pk[slot] && cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_pk[slot], 0) != cudaSuccess) return ST3_ERR_CUDA;
    if (cudaMemcpyAsync(dk, static_cast<const unsigned char*>(k_host) + (size_t)i * lp, lp, cudaMemcpyHostToDevice,
                        ctx->s_h2d) != cudaSuccess ||
        cudaMemcpyAsync(dv, static_cast<const unsigned char*>(v_host) + (size_t)i * lp, lp, cudaMemcpyHostToDevice,
                        ctx->s_h2d) != cudaSuccess ||
        cudaEventRecord(ctx->ev_pin[slot], ctx->s_h2d) != cudaSuccess ||
        cudaStreamWaitEvent(st, ctx->ev_pin[slot], 0) != cudaSuccess)
      return ST3_ERR_CUDA;
    const st3_status s = prefill_common(ctx, layer_begin + i, 1, dq + (size_t)i * lq, dk, dv, text_len, nullptr,
                                        dout + (size_t)i * lq, cuda_stream);
    if (s != ST3_OK) return s;
    if (cudaEventRecord(ctx->ev_pk[slot], st) != cudaSuccess) return ST3_ERR_CUDA;
    ctx->rec_pk[slot] = true;
    ctx->pseq++;
  }
  if (cudaEventRecord(ctx->ev_pq, st) != cudaSuccess) return ST3_ERR_CUDA;
  ctx->rec_pq = true;
  // the outputs of all layers in one copy, behind the last layer's kernels
  if (cudaMemcpyAsync(out_host, dout, lq * layer_count, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ST3_ERR_CUDA;
  return ST3_OK;
}

st3_status st3_host_sync(st3_ctx* ctx, void* cuda_stream) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  for (int i = 0; i < 2; ++i)
    if (ctx->rec_out[i] && cudaStreamWaitEvent(st, ctx->ev_out[i], 0) != cudaSuccess) return ST3_ERR_CUDA;
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
  if (cudaStreamSynchronize(ctx->last_stream) != cudaSuccess || cudaStreamSynchronize(ctx->s_h2d) != cudaSuccess ||
      cudaStreamSynchronize(ctx->s_d2h) != cudaSuccess)
    return ST3_ERR_CUDA;
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

st3_status st3_set_overlap(st3_ctx* ctx, int32_t on) {
  if (!ctx) return ST3_ERR_INVALID_ARG;
  ctx->overlap = on != 0;
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
  for (int i = 0; i < 2; ++i)
    for (cudaEvent_t e : {ctx->ev_in[i], ctx->ev_k[i], ctx->ev_out[i], ctx->ev_pin[i], ctx->ev_pk[i]})
      if (e) cudaEventDestroy(e);
  if (ctx->ev_pq) cudaEventDestroy(ctx->ev_pq);
  if (ctx->s_h2d) cudaStreamDestroy(ctx->s_h2d);
  if (ctx->s_d2h) cudaStreamDestroy(ctx->s_d2h);
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
