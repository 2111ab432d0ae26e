// Causal prompt attention (Eq. 2 in full) on the 5th-generation tensor cores: tcgen05.mma with
// accumulators in tensor memory, operands staged in shared memory by TMA, for bf16 and D = 128.
//
// One block per (head instance, 128-query tile), two blocks per SM.  Warp 4 is the control warp: it issues
// the TMA loads and the MMAs.  Warps 0-3 own one query row per thread (thread i <-> TMEM lane i), so the
// softmax needs no cross-thread reduction.  One pass over the 64-key tiles up to the diagonal, with an
// online softmax:
//   S = Q K^T (8 MMAs of 128x64x16) into one of two S tiles in tensor memory; P = exp2(S - ref) as bf16,
//   written over the first half of its S tile; O += P V (4 MMAs of 128x128x16, P read from tensor memory as
//   the A operand, accumulator in tensor memory).
// The tensor pipe runs S(0) S(1) | PV(0) S(2) | PV(1) S(3) | ...: the next tile's scores are ready before the
// softmax of this one ends, so the softmax warps wait for the tensor cores only to rescale O.  `ref` follows
// the row's running maximum lazily: O (and the running sum) are rescaled in tensor memory only when the
// maximum has grown by more than 2^8, so P never exceeds 256 and rescaling is rare after the first tiles; O
// is divided by the sum on the way out.  K tiles are fetched three ahead, V tiles two ahead.
// The last query row's logits on the visual positions are kept per head, normalised at the end and summed
// over heads by a second small kernel: the scores alpha (Sec. 3.2) that prune the NEXT layer.
//
// Shared-memory operand layout: 128-byte swizzle, K-major tiles of [rows][64 bf16] (what a TMA box with
// CU_TENSOR_MAP_SWIZZLE_128B writes); V is consumed as an MN-major B operand straight from the same
// kind of box.  Every wait is bounded; a timeout sets the error word and lets the block finish.
#include "st3_common.cuh"

#include <cuda.h>

namespace {

constexpr int kPfThreads = 160;       // 4 softmax warps + the control warp
constexpr int kTile = 128;            // queries per tile
constexpr int kKeys = 64;             // keys per tile
constexpr int kPfD = 128;
constexpr int kBoxBytes = 128 * 128;  // one TMA box of Q: 128 rows x 64 bf16
constexpr int kTileBytes2 = 2 * kBoxBytes;
constexpr int kKBoxBytes = kKeys * 128;  // one TMA box of K or V: 64 rows x 64 bf16
constexpr int kKTileBytes = 2 * kKBoxBytes;
constexpr uint32_t kTmemCols = 256;   // S in columns [0,64), O in [128,256)

// One box of [rows][64 bf16] of instance z, starting at row y (may be negative or reach past the instance's
// last row: such rows are filled with zeros, never with a neighbouring instance's data) and column x (0 or 64).
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_cta(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait; false after ~2 s (the caller sets the error word and stops issuing work).
__device__ __forceinline__ bool pf_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
// The whole warp waits and takes the same verdict: the tensor-memory accesses and __syncwarp that follow a wait
// are warp-wide, so a timeout must not split the warp.
__device__ __forceinline__ bool pf_wait_warp(uint64_t* bar, uint32_t parity) {
  return __all_sync(0xffffffffu, pf_wait(bar, parity));
}
// Shared-memory matrix descriptors: 128-byte swizzle, 8-row groups 1024 bytes apart.
// The descriptor's high word is the same for every operand here; the low word is the address field plus the
// leading-dimension byte offset, so stepping through a tile is one 32-bit add (shared addresses stay below
// 2^18, i.e. inside the 14-bit field, whatever is added).
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3fffu) | ((lbo_bytes >> 4) << 16);
}
// One MMA step (K = 16): D[tmem_d] (+)= A * B with both operands in shared memory.  `accumulate` is a
// compile-time constant or a value fixed for the tile at every call site.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, {%5, %5, %5, %5}, p;\n\t}"
      :
      : "r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(0u), "r"(kDescHi)
      : "memory");
}
// the same with the A operand in tensor memory (lane = row, two bf16 per 32-bit column along K)
__device__ __forceinline__ void umma_bf16_ta(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_lo, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, {%5, %5, %5, %5}, p;\n\t}"
      :
      : "r"(tmem_d), "r"(tmem_a), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(0u), "r"(kDescHi)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 64 consecutive columns of this thread's lane in one instruction (one round trip instead of two)
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]),
        "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]),
        "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]),
        "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]),
        "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
  u64 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// kind::f16 instruction descriptors: fp32 accumulate, bf16 x bf16, M = 128.
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);
constexpr uint32_t kIdescS = kIdescBase | ((kKeys >> 3) << 17);                 // N = 64 keys, A and B K-major
constexpr uint32_t kIdescPV = kIdescBase | ((128u >> 3) << 17) | (1u << 16);    // N = 128 dims, B (= V) MN-major

struct PfShared {   // after the tiles in dynamic shared memory
  uint64_t bar_q, bar_k[3], bar_v[2], bar_s[2], bar_p[2], bar_o, bar_done;
  uint32_t tmem;
  int fail;
  float last[2];
};
constexpr int kPfSmem = kTileBytes2 + 5 * kKTileBytes + 128;   // Q, two V and three K buffers, PfShared
static_assert(sizeof(PfShared) <= 128, "PfShared must fit its slot");

struct PrefillParams {
  __nv_bfloat16* out;   // [num_inst][T][128]
  float* head_probs;    // [num_inst][num_visual] last-row probabilities per head
  int* status;          // error word (may be null)
  int T, sys_len, num_visual;
};

__global__ void __launch_bounds__(kPfThreads, 2)
st3_prefill_attend_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                          const __grid_constant__ CUtensorMap map_v, const PrefillParams p) {
  // Two blocks per SM leave each 113 KB: the tiles take 112 KB of it, so there is no room for alignment slack.
  // The kernel has no static shared memory, which puts the dynamic window at the (1024-byte aligned) start of
  // the block's allocation; the tiles come first and the small variables after them.  A misaligned window is
  // reported, not used (the 128-byte swizzle of TMA and of the MMA descriptors assumes 1024-byte aligned tiles).
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem;
  unsigned char* sV2 = sQ + kTileBytes2;      // two V buffers: tile t+2 replaces tile t once P V(t) is complete
  unsigned char* sK2 = sV2 + 2 * kKTileBytes; // three K buffers: tile t+3 replaces tile t once S(t) is complete
  PfShared& sh = *reinterpret_cast<PfShared*>(sK2 + 3 * kKTileBytes);
  uint64_t &bar_q = sh.bar_q, &bar_o = sh.bar_o, &bar_done = sh.bar_done;
  uint64_t (&bar_p)[2] = sh.bar_p;
  uint64_t (&bar_k)[3] = sh.bar_k;
  uint64_t (&bar_v)[2] = sh.bar_v, (&bar_s)[2] = sh.bar_s;
  uint32_t& s_tmem = sh.tmem;
  int& s_fail = sh.fail;
  float (&s_last)[2] = sh.last;
  if (smem_u32(smem) & 1023u) {
    if (threadIdx.x == 0 && p.status) atomicOr(p.status, ST3_DEV_RANGE);
    return;
  }

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x, inst = blockIdx.y;   // an instance's longest causal prefixes start first
  const int T = p.T;
  const int row_base = inst * T;  // first row of this instance in the [num_inst * T][128] tensors
  // Query tiles are aligned to the END of the prompt: the ragged tile is the first one, where the causal prefix
  // is shortest, instead of the last one, where a mostly empty tile would walk every key.  Its rows before the
  // prompt (q0 < 0) are dead: their loads read the fill value (zeros), nothing is stored.
  const int q0 = T - ((int)gridDim.x - qt) * kTile;                // first query row of this tile
  const int nkt = (q0 + kTile + kKeys - 1) / kKeys;                // causal: key tiles up to the diagonal

  if (tid == 4 * 32) {   // the control warp's first lane: barriers, then the first loads at once (they are in
                         // flight during the rest of the set-up)
    mbar_init(&bar_q, 1); mbar_init(&bar_k[0], 1); mbar_init(&bar_k[1], 1); mbar_init(&bar_k[2], 1); mbar_init(&bar_v[0], 1); mbar_init(&bar_v[1], 1);
    mbar_init(&bar_s[0], 1); mbar_init(&bar_s[1], 1); mbar_init(&bar_o, 1);
    mbar_init(&bar_p[0], 128); mbar_init(&bar_p[1], 128); mbar_init(&bar_done, 1);
    s_fail = 0;
    mbar_fence_init();
    mbar_expect_tx(&bar_q, kTileBytes2);
    tma_load_3d(sQ, &map_q, 0, q0, inst, &bar_q);
    tma_load_3d(sQ + kBoxBytes, &map_q, 64, q0, inst, &bar_q);
    for (int kt = 0; kt < 3 && kt < nkt; ++kt) {
      unsigned char* d = sK2 + kt * kKTileBytes;
      mbar_expect_tx(&bar_k[kt], kKTileBytes);
      tma_load_3d(d, &map_k, 0, kt * kKeys, inst, &bar_k[kt]);
      tma_load_3d(d + kKBoxBytes, &map_k, 64, kt * kKeys, inst, &bar_k[kt]);
    }
    for (int kt = 0; kt < 2 && kt < nkt; ++kt) {
      unsigned char* d = sV2 + kt * kKTileBytes;
      mbar_expect_tx(&bar_v[kt], kKTileBytes);
      tma_load_3d(d, &map_v, 0, kt * kKeys, inst, &bar_v[kt]);
      tma_load_3d(d + kKBoxBytes, &map_v, 64, kt * kKeys, inst, &bar_v[kt]);
    }
  }
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t tmem_O = tmem + 128;   // S(t) lives at column 64 * (t & 1)
  volatile int* fail = &s_fail;

  if (warp == 4) {
    // ===================== control warp =====================
    // Tensor-pipe order: S(0) S(1) | PV(0) S(2) | PV(1) S(3) | ...  -- S(t+1) is already in tensor memory when
    // the softmax of tile t ends, so the softmax warps never wait for the tensor cores in steady state.
    bool ok = true;
    auto load_k = [&](int kt) {
      unsigned char* d = sK2 + (kt % 3) * kKTileBytes;
      mbar_expect_tx(&bar_k[kt % 3], kKTileBytes);
      tma_load_3d(d, &map_k, 0, kt * kKeys, inst, &bar_k[kt % 3]);
      tma_load_3d(d + kKBoxBytes, &map_k, 64, kt * kKeys, inst, &bar_k[kt % 3]);
    };
    auto load_v = [&](int kt) {
      unsigned char* d = sV2 + (kt & 1) * kKTileBytes;
      mbar_expect_tx(&bar_v[kt & 1], kKTileBytes);
      tma_load_3d(d, &map_v, 0, kt * kKeys, inst, &bar_v[kt & 1]);
      tma_load_3d(d + kKBoxBytes, &map_v, 64, kt * kKeys, inst, &bar_v[kt & 1]);
    };
    // S(kt) = Q K(kt)^T: 8 steps of 16 along the head dimension
    const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), k_lo = desc_lo(smem_u32(sK2), 16);
    const uint32_t v_lo = desc_lo(smem_u32(sV2), kKBoxBytes);
    auto issue_s = [&](int kt) {
      const uint32_t kb = k_lo + (uint32_t)(kt % 3) * (kKTileBytes >> 4);
      const uint32_t tmem_S = tmem + (uint32_t)(kt & 1) * kKeys;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t offq = (ks >> 2) * kBoxBytes + (ks & 3) * 32;
        const uint32_t offk = (ks >> 2) * kKBoxBytes + (ks & 3) * 32;
        umma_bf16(tmem_S, q_lo + (offq >> 4), kb + (offk >> 4), kIdescS, ks > 0);
      }
      umma_commit(&bar_s[kt & 1]);
    };
    ok = pf_wait_warp(&bar_q, 0);   // (Q, K(0..2) and V(0..1) were requested during the set-up)
    // prologue: S(0) and S(1)
    for (int kt = 0; kt < 2 && kt < nkt && ok; ++kt) {
      ok = pf_wait_warp(&bar_k[kt], 0);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) issue_s(kt);
      __syncwarp();
    }
    for (int kt = 0; kt < nkt && ok; ++kt) {
      // P(kt) is in tensor memory, so S(kt) is complete and K(kt)'s buffer is free: K(kt+3) goes there
      ok = pf_wait_warp(&bar_p[kt & 1], (kt >> 1) & 1);
      if (!ok) break;
      if (lane == 0 && kt + 3 < nkt) load_k(kt + 3);
      __syncwarp();
      ok = pf_wait_warp(&bar_v[kt & 1], (kt >> 1) & 1);   // V(kt) has landed
      if (!ok) break;
      if (kt + 2 < nkt) { ok = pf_wait_warp(&bar_k[(kt + 2) % 3], ((kt + 2) / 3) & 1); if (!ok) break; }
      tc_fence_after();
      if (lane == 0) {
        // O += P V: 4 steps of 16 keys; P is read from tensor memory, where it replaced the first half of its
        // S tile (8 columns per 16 keys); V is the MN-major operand (two 64-dim boxes 8 KB apart)
        const uint32_t vb = v_lo + (uint32_t)(kt & 1) * (kKTileBytes >> 4);
        const uint32_t tmem_P = tmem + (uint32_t)(kt & 1) * kKeys;
#pragma unroll
        for (int ks = 0; ks < kKeys / 16; ++ks)
          umma_bf16_ta(tmem_O, tmem_P + ks * 8, vb + ks * (2048 >> 4), kIdescPV, (kt > 0 || ks > 0));
        umma_commit(&bar_o);
        if (kt == nkt - 1) umma_commit(&bar_done);   // O is complete
        if (kt + 2 < nkt) issue_s(kt + 2);   // into the S buffer whose tile the softmax warps have just left
      }
      __syncwarp();
      // V(kt)'s buffer is free once P V(kt) is complete: V(kt+2) goes there
      ok = pf_wait_warp(&bar_o, kt & 1);
      if (!ok) break;
      if (lane == 0 && kt + 2 < nkt) load_v(kt + 2);
      __syncwarp();
    }
    if (!ok) { *fail = 1; if (lane == 0 && p.status) atomicOr(p.status, ST3_DEV_COPY_TIMEOUT); }
  } else {
    // ===================== softmax warps: thread <-> query row =====================
    const int r = tid;                        // row inside the tile == TMEM lane
    const int qi = q0 + r;                    // query position inside the instance (< T always)
    const bool live = qi >= 0;
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    const float sc = 1.4426950408889634f * rsqrtf((float)kPfD);
    float ref = -INFINITY;   // what P is taken relative to; trails the running maximum by at most 8 (log2 domain)
    float l = 0.f;           // running sum of exp2(s - ref)
    bool ok = true;
    float* probs = p.head_probs ? p.head_probs + (size_t)inst * p.num_visual : nullptr;
    const bool last_row = live && qi == T - 1;
    for (int kt = 0; kt < nkt && ok; ++kt) {
      ok = pf_wait_warp(&bar_s[kt & 1], (kt >> 1) & 1);   // a failed control warp stops issuing: this wait then runs out
      if (!ok) break;
      tc_fence_after();
      const uint32_t tmem_S = tmem + (uint32_t)(kt & 1) * kKeys;
      uint32_t v[64];
      tmem_ld64(tmem_S + lane_addr, v);
      const int j0 = kt * kKeys;
      if (j0 + kKeys > q0 + 1) {   // the tile reaches past the first row's own position: mask (also covers keys >= T)
#pragma unroll
        for (int c = 0; c < 64; ++c)
          if (!(live && j0 + c <= qi && j0 + c < T)) v[c] = 0xff800000u;
      }
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 64; c += 8)
#pragma unroll
        for (int e = 0; e < 4; ++e) m4[e] = fmax3(m4[e], __uint_as_float(v[c + e]), __uint_as_float(v[c + 4 + e]));
      const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * sc;   // the scale is positive: max and scaling commute
      if (probs && qt == (int)gridDim.x - 1 && warp == 3) {
        // the last query row lives in one lane of this warp: hand its logits on the visual positions to the
        // whole warp, which stores them coalesced; they are normalised once the row is complete
        const int src = 31;   // the last query row is the last row of the last tile
#pragma unroll
        for (int c = 0; c < 64; c += 32) {
          float mine = 0.f;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float x = __shfl_sync(0xffffffffu, __uint_as_float(v[c + e]), src);
            if (lane == e) mine = x;
          }
          const int ja = j0 + c + lane - p.sys_len;
          if (ja >= 0 && ja < p.num_visual) probs[ja] = mine * sc;
        }
      }
      // lazy rescale: move the reference only when the maximum has run away from it
      float factor = 1.f;
      if (mx > ref + 8.f) {
        factor = ref > -INFINITY ? fast_exp2(ref - mx) : 0.f;
        ref = mx;
      }
      l *= factor;
      // probabilities exp2(s * sc - ref) as packed bf16 pairs (exp2(-inf) = 0 for masked keys); the scaling runs
      // as packed two-wide FMAs
      const float nrf = ref > -INFINITY ? -ref : 0.f;   // a row with no key yet (padding rows) yields zeros
      const u64 sc2 = pack2(sc, sc), nrf2 = pack2(nrf, nrf);
      u64 add[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};   // row sum, as two packed pairs
      uint32_t w[32];
#pragma unroll
      for (int c = 0; c < 64; c += 2) {
        u64 t2 = nrf2;
        fma2(t2, pack2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), sc2);
        float ta, tb;
        split2(t2, ta, tb);
        const float pa = fast_exp2(ta), pb = fast_exp2(tb);
        add[(c >> 1) & 1] = add2(add[(c >> 1) & 1], pack2(pa, pb));
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(pa, pb);
        w[c >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
      }
      l += sum2(add2(add[0], add[1]));
      // P V(kt-1) must be complete before O is rescaled in place; only then is it waited for.  The parity wait is
      // unambiguous although this thread has not watched every phase: S(kt) is complete, hence so is P V(kt-2),
      // issued before it, and P V(kt) cannot be issued before this thread's arrival below, so the barrier is in
      // phase kt-1 or has just left it.
      if (kt > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
        ok = pf_wait_warp(&bar_o, (kt - 1) & 1);
        if (!ok) break;
        tc_fence_after();
        {
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            uint32_t o[32];
            tmem_ld32(tmem_O + lane_addr + cb * 32, o);
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * factor);
            tmem_st32(tmem_O + lane_addr + cb * 32, o);
          }
        }
      }
      // P replaces the first 32 columns of this S tile (only this thread reads or writes this lane of it, and
      // S(kt+2) lands there after P V(kt) in the tensor pipe's order)
      // Arrivals alternate between two barriers: a thread one tile ahead of the slowest one (it cannot be further,
      // S(kt+2) is issued only after every arrival for tile kt) then never adds to the slow one's phase.
      tmem_st32(tmem_S + lane_addr, w);
      tc_fence_before();
      mbar_arrive_cta(&bar_p[kt & 1]);
    }
    if (ok) { ok = pf_wait_warp(&bar_done, 0) && !*fail; }   // the last P V: O is complete
    const float inv_l = l > 0.f ? 1.f / l : 0.f;
    if (probs && qt == (int)gridDim.x - 1) {   // this block holds the last query row (same answer in every thread)
      // alpha of this head: exp2(logit - ref) / sum over the visual positions, with the last row's final
      // reference and sum; the 128 softmax threads share the work
      if (last_row) { s_last[0] = ref; s_last[1] = ok ? inv_l : 0.f; }
      __threadfence_block();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      const float rl = s_last[0], il = s_last[1];
      for (int i = tid; i < p.num_visual; i += 128) probs[i] = fast_exp2(probs[i] - rl) * il;
    }
    // ---- O / sum -> bf16 -> global ----
    if (ok) {
      tc_fence_after();
      __nv_bfloat16* orow = p.out + ((size_t)row_base + qi) * kPfD;
#pragma unroll 1
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_O + lane_addr + cb * 32, v);
        if (live) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[c + 2 * e]) * inv_l,
                                                              __uint_as_float(v[c + 2 * e + 1]) * inv_l);
              w[e] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(orow + cb * 32 + c) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// scores[b][i] = sum over the heads of sequence b of the last row's probability on visual token i
__global__ void st3_prefill_scores_kernel(const float* __restrict__ head_probs, float* __restrict__ scores, int num_heads,
                                          int num_visual) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= num_visual) return;
  float s = 0.f;
  for (int h = 0; h < num_heads; ++h) s += head_probs[((size_t)b * num_heads + h) * num_visual + i];
  scores[(size_t)b * num_visual + i] = s;
}

// The same sum for a layer that ran on the visual tokens an earlier layer kept: position i of the layer's visual
// span is original token ids[b][i], and the scores go out indexed by original token (tokens not held: -1).
__global__ void st3_prefill_fill_kernel(float* __restrict__ scores, long long n, float value) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) scores[i] = value;
}
__global__ void st3_prefill_scores_by_id_kernel(const float* __restrict__ head_probs, const int* __restrict__ ids,
                                                float* __restrict__ scores, int* status, int num_heads, int num_visual,
                                                int num_visual_total) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= num_visual) return;
  const int id = ids[(size_t)b * num_visual + i];
  if ((unsigned)id >= (unsigned)num_visual_total) {  // reported, not used
    if (status) atomicOr(status, ST3_DEV_RANGE);
    return;
  }
  float s = 0.f;
  for (int h = 0; h < num_heads; ++h) s += head_probs[((size_t)b * num_heads + h) * num_visual + i];
  scores[(size_t)b * num_visual_total + id] = s;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [num_inst][rows][128] bf16 tensor, boxes of box_rows rows x 64 columns inside one instance, 128-byte swizzle;
// rows outside [0, rows) of the instance read as zero, so a tile at the end of one instance never sees the next.
bool make_map(EncodeTiledFn fn, CUtensorMap* map, const void* base, size_t num_inst, size_t rows, int box_rows) {
  const cuuint64_t dims[3] = {128, (cuuint64_t)rows, (cuuint64_t)num_inst};
  const cuuint64_t strides[2] = {256, (cuuint64_t)rows * 256};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

static st3_status prefill_attend_impl(const void* q, const void* k, const void* v, void* out, float* head_probs,
                                      float* scores, int* dev_status, int32_t num_inst, int32_t num_heads,
                                      int32_t seq_len, int32_t head_dim, int32_t dtype, int32_t sys_len,
                                      int32_t num_visual, const int32_t* ids, int32_t num_visual_total,
                                      void* cuda_stream) {
  auto aligned = [](const void* ptr) { return ptr && (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; };
  if (!aligned(q) || !aligned(k) || !aligned(v) || !aligned(out)) return ST3_ERR_INVALID_ARG;
  if (num_inst < 1 || num_heads < 1 || num_inst % num_heads || seq_len < 1) return ST3_ERR_INVALID_ARG;
  if (sys_len < 0 || num_visual < 0 || sys_len + num_visual > seq_len) return ST3_ERR_INVALID_ARG;
  if (num_visual > 0 && (!head_probs || !scores)) return ST3_ERR_INVALID_ARG;
  if (head_dim != kPfD || dtype != ST3_BF16) return ST3_ERR_UNSUPPORTED;
  if ((long long)num_inst * seq_len > 0x7fffffffLL || num_inst > 65535) return ST3_ERR_UNSUPPORTED;
  // looked up once (initialisation of a local static is thread-safe); null if the driver does not offer it
  static const EncodeTiledFn encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      fn = nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
  }();
  if (!encode) return ST3_ERR_CUDA;
  CUtensorMap mq, mk, mv;
  if (!make_map(encode, &mq, q, (size_t)num_inst, (size_t)seq_len, kTile) ||
      !make_map(encode, &mk, k, (size_t)num_inst, (size_t)seq_len, kKeys) ||
      !make_map(encode, &mv, v, (size_t)num_inst, (size_t)seq_len, kKeys))
    return ST3_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int smem = kPfSmem;
  if (cudaFuncSetAttribute(st3_prefill_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return ST3_ERR_CUDA;
  PrefillParams p;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.head_probs = num_visual > 0 ? head_probs : nullptr;
  p.status = dev_status;
  p.T = seq_len; p.sys_len = sys_len; p.num_visual = num_visual;
  const dim3 grid((unsigned)((seq_len + kTile - 1) / kTile), (unsigned)num_inst);
  st3_prefill_attend_kernel<<<grid, kPfThreads, smem, st>>>(mq, mk, mv, p);
  const int num_seq = num_inst / num_heads;
  if (ids) {
    const long long n = (long long)num_seq * num_visual_total;
    st3_prefill_fill_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(scores, n, -1.f);
    if (num_visual > 0) {
      const dim3 g2((unsigned)((num_visual + 255) / 256), (unsigned)num_seq);
      st3_prefill_scores_by_id_kernel<<<g2, 256, 0, st>>>(head_probs, ids, scores, dev_status, num_heads, num_visual,
                                                          num_visual_total);
    }
  } else if (num_visual > 0) {
    const dim3 g2((unsigned)((num_visual + 255) / 256), (unsigned)num_seq);
    st3_prefill_scores_kernel<<<g2, 256, 0, st>>>(head_probs, scores, num_heads, num_visual);
  }
  return cudaGetLastError() == cudaSuccess ? ST3_OK : ST3_ERR_CUDA;
}

extern "C" st3_status st3_prefill_attend(const void* q, const void* k, const void* v, void* out, float* head_probs,
                                         float* scores, int* dev_status, int32_t num_inst, int32_t num_heads,
                                         int32_t seq_len, int32_t head_dim, int32_t dtype, int32_t sys_len,
                                         int32_t num_visual, void* cuda_stream) {
  return prefill_attend_impl(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len, head_dim,
                             dtype, sys_len, num_visual, nullptr, 0, cuda_stream);
}

extern "C" st3_status st3_prefill_attend_kept(const void* q, const void* k, const void* v, void* out,
                                              float* head_probs, float* scores, int* dev_status, int32_t num_inst,
                                              int32_t num_heads, int32_t seq_len, int32_t head_dim, int32_t dtype,
                                              int32_t sys_len, int32_t num_visual, const int32_t* ids,
                                              int32_t num_visual_total, void* cuda_stream) {
  if (!ids || (reinterpret_cast<uintptr_t>(ids) & 3u) || !scores || num_visual_total < num_visual ||
      num_visual_total < 1)
    return ST3_ERR_INVALID_ARG;
  return prefill_attend_impl(q, k, v, out, head_probs, scores, dev_status, num_inst, num_heads, seq_len, head_dim,
                             dtype, sys_len, num_visual, ids, num_visual_total, cuda_stream);
}
