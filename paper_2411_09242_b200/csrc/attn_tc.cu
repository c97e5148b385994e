// Fused attention for sm_100a: S = Q.K^T and O = softmax(S).V on tcgen05 tensor cores with the
// score tiles kept in tensor memory; the [S, S] score / probability tensors never reach HBM or the
// arena. Two forms. Sequences of more than one query tile run the persistent two-tile form described further down
// (probabilities stay in tensor memory). The one-tile form, described here, serves sequences of a single query tile
// and A/B timing: one CTA = one (batch, head, 128-query tile); 320 threads: 8 softmax warps (two threads per
// query row, 64 key columns each), one warp that issues the MMAs, one warp that issues the TMA loads.
// (Sixteen softmax warps, four threads per row, were measured and are no faster: with 128 x 128 x 16 and
// 128 x D x 16 instructions costing the same ~128 cycles as a 128 x 256 x 16 one, the tensor pipe is
// busy ~1500-2000 of the ~2400 cycles a key tile takes.)
//
//   per 128-key tile:  TMA K, V tiles (2-stage rings)  ->  tcgen05.mma  S = Q.K^T  (one of two TMEM tiles, fp32)
//                      -> tcgen05.ld, online softmax in registers (row max / sum per thread, exp2)
//                      -> P (bf16) written to one of two shared-memory tiles, 128-byte-swizzled K-major
//                      -> tcgen05.mma  O += P.V (TMEM; rescaled in place only when the row maximum jumps)
//
// Q, K and V are read where the plan put them: Q with the head dim contiguous; K either with the
// head dim contiguous (any of the [B,S,nh,D] / [B,nh,S,D] families) or sequence-contiguous
// ([B,nh,D,S]); V likewise. The TMA boxes and the shared-memory matrix descriptors follow the
// operand's major, as in the GEMM kernel. No cluster multicast. All waits are bounded.
#include <cuda.h>

#include <algorithm>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

constexpr int TQ = 128;   // queries per CTA
constexpr int TK = 128;   // keys per step
constexpr long long kWaitCycles = 3000000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255) == 0 && clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ __forceinline__ void tma_load5(uint32_t dst, const CUtensorMap* map, uint32_t bar, const int* c) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4])
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// Descriptors given as 32-bit halves: only the low word (the address field) differs between the MMAs of a tile.
__device__ __forceinline__ void umma_bf16_lohi(uint32_t tmem_c, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                               uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n .reg .b64 da, db;\n mov.b64 da, {%1, %2};\n mov.b64 db, {%3, %4};\n setp.ne.b32 p, %6, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}"
      ::"r"(tmem_c), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 128-byte-swizzled shared-memory matrix descriptor; lbo/sbo in bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return uint64_t((saddr & 0x3FFFF) >> 4) | (uint64_t(lbo >> 4) << 16) | (uint64_t(sbo >> 4) << 32) |
         (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
__device__ __forceinline__ uint32_t make_idesc(int n, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn) << 15) | (uint32_t(b_mn) << 16) |
         (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

// bz = batch * heads + head is split as (bz / b0, bz % b0): b0 = heads when the two strides do not
// chain, b0 = batch * heads (one merged dim) when they do
__device__ __forceinline__ void coords(const int* sel, int k, int r, int bz, int b0, int* c) {
  const int lo = bz % b0, hi = bz / b0;
#pragma unroll
  for (int d = 0; d < 5; ++d) {
    const int q = sel[d];
    c[d] = q == 0 ? k : q == 2 ? r : q == 4 ? lo : q == 5 ? hi : 0;
  }
}

__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&q)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]), "r"(q[4]), "r"(q[5]), "r"(q[6]),
      "r"(q[7]), "r"(q[8]), "r"(q[9]), "r"(q[10]), "r"(q[11]), "r"(q[12]), "r"(q[13]), "r"(q[14]), "r"(q[15]),
      "r"(q[16]), "r"(q[17]), "r"(q[18]), "r"(q[19]), "r"(q[20]), "r"(q[21]), "r"(q[22]), "r"(q[23]), "r"(q[24]),
      "r"(q[25]), "r"(q[26]), "r"(q[27]), "r"(q[28]), "r"(q[29]), "r"(q[30]), "r"(q[31])
      : "memory");
}

constexpr int kSoftmaxThreads = 256;
#ifndef FLUID_ATTN_POLY_EVERY
#define FLUID_ATTN_POLY_EVERY 0
#endif
// One pair of exponentials in this many goes to the fused-multiply-add pipe instead of the special-function unit (0: none).
// Measured with a share of 1/4 and 1/2: slower (2 x 4096 x 32 x 128: 918 -> 807 -> 652 TFLOP/s): a softmax warp is bound by
// the instructions it can issue alone on its scheduler, not by the special-function unit, and the polynomial costs 8.
constexpr int kPolyEvery = FLUID_ATTN_POLY_EVERY;
constexpr int kAttnThreads = kSoftmaxThreads + 64;   // warps 0-7 softmax (two threads per query row), warp 8 MMAs, warp 9 loads

// Warps 0-7: softmax. Warp 8, one thread: every tcgen05.mma. Warp 9: TMA loads. They meet only at mbarriers:
//   s_full[i]  S tile i (of two, in tensor memory) holds Q.K_j^T          MMA commit -> softmax
//   p_full[i]  P tile i (of two, in shared memory) is written and S tile i is read    256 softmax threads -> MMA
//   o_done[i]  P_j.V_j has been accumulated into O (j odd / even)         MMA commit -> softmax (rescale, P reuse, end)
//   k_full[i], v_full[i]  K / V stage i has landed                        TMA -> MMA
// (the loader reuses a K stage when s_full says its Q.K^T has run, a V stage when o_done says its P.V has)
// so the tensor core works on Q.K_{j+2}^T and P_j.V_j while the softmax warps are on tile j+1.
template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const __grid_constant__ AttnParams p) {
  constexpr int DC = D / 64;                       // 64-wide chunks of the head dim
  constexpr uint32_t kTile = TQ * D * 2;           // bytes of one Q / K / V tile
  constexpr uint32_t kPBytes = TQ * TK * 2;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = raw;                       // 1024-byte aligned (checked below): the tiles leave no slack for rounding
  const uint32_t sQ = base, sK = sQ + kTile, sV = sK + 2 * kTile, sP = sV + 2 * kTile, bars = sP + 2 * kPBytes;
  const uint32_t bar_q = bars, k_full = bars + 8, v_full = bars + 24, s_full = bars + 40, p_full = bars + 56, o_done = bars + 72;
  const uint32_t tmem_slot = bars + 88;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  volatile uint32_t* abort_flag = tmem_slot_ptr + 1;
  float* xch = reinterpret_cast<float*>(smem_raw + (bars + 128 - raw));   // [2 tiles][2 halves][128 rows]
  uint8_t* p_smem = smem_raw + (sP - raw);

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5;
  // CTAs are issued heaviest first: with a causal mask the last query tiles see the most key tiles,
  // so they start first and the short ones fill the gaps (longest-processing-time order)
  const int n_bz = p.B * p.NH;
  const int mt = (int(gridDim.x) / n_bz - 1) - int(blockIdx.x) / n_bz, bz = int(blockIdx.x) % n_bz;
  const int h = bz % p.NH, b = bz / p.NH;
  const int m0 = mt * TQ;
  int n_kv = (p.S + TK - 1) / TK;
  if (p.causal) n_kv = min(n_kv, (m0 + TQ - 1) / TK + 1);
  if (raw & 1023u) {   // cannot happen with the launch this file does; refuse rather than run misaligned tiles
    if (threadIdx.x == 0) atomicOr(p.status, 0x100u | 0x08u);
    return;
  }

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(k_full + 8 * i, 1); mbar_init(v_full + 8 * i, 1); mbar_init(s_full + 8 * i, 1);
      mbar_init(p_full + 8 * i, kSoftmaxThreads); mbar_init(o_done + 8 * i, 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  const uint32_t tS = tmem_base, tO = tmem_base + 2 * TK;     // two score tiles, then the output accumulator

  if (warp == 9) {
    // ======================= loads =======================
    // Lane 0 does every wait. The TMA boxes of a K or V tile (four for D = 128, two for D = 64) each
    // belong to one lane, which keeps that box's coordinates in registers and advances them by one key
    // tile per load: the divisions and selects behind a coordinate are done once.
    const int lane = threadIdx.x & 31;
    const bool lead = lane == 0;
    constexpr int NB = 2 * DC;               // boxes per tile
    const bool k_lane = lane < NB, v_lane = lane >= NB && lane < 2 * NB;
    const int bx = k_lane ? lane : lane - NB;
    int cur[5] = {0, 0, 0, 0, 0}, inc[5] = {0, 0, 0, 0, 0};
    uint32_t box_dst = 0;
    if (k_lane) {
      if (!p.k_mn_major) {          // [d chunk][128 keys][64 d]: box (dc, rh)
        const int dc = bx >> 1, rh = bx & 1;
        coords(p.k_sel, dc * 64, rh * 64, bz, p.k_b0, cur);
        box_dst = sK + dc * 16384u + rh * 8192u;
      } else {                      // [key chunk][D d-rows][64 keys]: box (sc, dc)
        const int sc = bx / DC, dc = bx % DC;
        coords(p.k_sel, dc * 64, sc * 64, bz, p.k_b0, cur);
        box_dst = sK + sc * (D * 128u) + dc * 8192u;
      }
#pragma unroll
      for (int d = 0; d < 5; ++d) inc[d] = p.k_sel[d] == 2 ? TK : 0;   // the key index is K's row index
    } else if (v_lane) {
      if (!p.v_k_major) {           // [d chunk][128 keys][64 d]  (MN-major B of P.V): box (dc, kc)
        const int dc = bx >> 1, kc = bx & 1;
        coords(p.v_sel, kc * 64, dc * 64, bz, p.v_b0, cur);
        box_dst = sV + dc * 16384u + kc * 8192u;
      } else {                      // [key chunk][D d-rows][64 keys]  (K-major B of P.V): box (kc, dh)
        const int kc = bx / DC, dh = bx % DC;
        coords(p.v_sel, kc * 64, dh * 64, bz, p.v_b0, cur);
        box_dst = sV + kc * (D * 128u) + dh * 8192u;
      }
#pragma unroll
      for (int d = 0; d < 5; ++d) inc[d] = p.v_sel[d] == 0 ? TK : 0;   // the key index is V's contraction index
    }
    uint32_t fail = 0;
    int k_issued = 0, v_issued = 0;   // tiles whose loads have been issued (uniform across the warp)
    auto load_k = [&](int j) {        // called by the whole warp
      const uint32_t bar = k_full + 8u * (j & 1);
      if (lead) mbar_expect_tx(bar, kTile);
      if (k_lane) {
        tma_load5(box_dst + uint32_t(j & 1) * kTile, &map_k, bar, cur);
#pragma unroll
        for (int d = 0; d < 5; ++d) cur[d] += inc[d];
      }
      k_issued = j + 1;
    };
    auto load_v = [&](int j) {
      const uint32_t bar = v_full + 8u * (j & 1);
      if (lead) mbar_expect_tx(bar, kTile);
      if (v_lane) {
        tma_load5(box_dst + uint32_t(j & 1) * kTile, &map_v, bar, cur);
#pragma unroll
        for (int d = 0; d < 5; ++d) cur[d] += inc[d];
      }
      v_issued = j + 1;
    };
    auto all_ok = [&](bool mine) { return __shfl_sync(0xffffffffu, mine ? 1 : 0, 0) != 0; };   // lane 0 decides; also re-converges the warp

    // the Q boxes' coordinates are index arithmetic: ready before the wait for the previous step
    int qc[2 * DC][5];
    if (lead) {
#pragma unroll
      for (int dc = 0; dc < DC; ++dc)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) coords(p.q_sel, dc * 64, m0 + rh * 64, bz, p.q_b0, qc[dc * 2 + rh]);
    }
    pdl_wait();  // Q, K, V come from the previous steps
    if (lead) {
      mbar_expect_tx(bar_q, kTile);
#pragma unroll
      for (int dc = 0; dc < DC; ++dc)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) tma_load5(sQ + dc * 16384u + rh * 8192u, &map_q, bar_q, qc[dc * 2 + rh]);
    }
    load_k(0);
    if (n_kv > 1) load_k(1);
    load_v(0);
    if (n_kv > 1) load_v(1);
    bool ok = true;
    for (int j = 0; ok && j + 2 < n_kv; ++j) {
      const int st = j & 1;
      const uint32_t ph = uint32_t(j >> 1) & 1u;
      // K stage st is free once Q.K_j^T has run
      if (lead && !mbar_wait(s_full + 8u * st, ph)) { fail |= 0x40u; ok = false; }
      ok = all_ok(ok);
      if (!ok) break;
      load_k(j + 2);
      // V stage st is free once P_j.V_j has run
      if (lead && !mbar_wait(o_done + 8u * st, ph)) { fail |= 0x80u; ok = false; }
      ok = all_ok(ok && !*abort_flag);
      if (!ok) break;
      load_v(j + 2);
    }
    if (!ok && lead) {
      *abort_flag = 1;
      if (fail) atomicOr(p.status, 0x100u | fail);
    }
    if (lead && *abort_flag) {
      // let loads still in flight land before the shared memory is given up (each wait is bounded)
      for (int j = max(0, k_issued - 2); j < k_issued; ++j) mbar_wait(k_full + 8u * (j & 1), uint32_t(j >> 1) & 1u);
      for (int j = max(0, v_issued - 2); j < v_issued; ++j) mbar_wait(v_full + 8u * (j & 1), uint32_t(j >> 1) & 1u);
    }
  } else if (warp == 8) {
    // ======================= MMAs (one thread) =======================
    if (threadIdx.x == kSoftmaxThreads) {
      uint32_t fail = 0;
      const uint32_t idesc_s = make_idesc(TK, 0, p.k_mn_major);
      const uint32_t idesc_o = make_idesc(D, 0, p.v_k_major ? 0 : 1);
      // descriptor halves: the high word is fixed per operand kind, the low word is base + a per-slice
      // offset (16-byte units) + the stage offset
      const uint64_t dq = make_desc(sQ, 16, 1024);
      const uint64_t dk = p.k_mn_major ? make_desc(sK, D * 128u, 1024) : make_desc(sK, 16, 1024);
      const uint64_t dp = make_desc(sP, 16, 1024);
      const uint64_t dv = p.v_k_major ? make_desc(sV, 16, 1024) : make_desc(sV, 16384, 1024);
      const uint32_t q_hi = uint32_t(dq >> 32), k_hi = uint32_t(dk >> 32), p_hi = uint32_t(dp >> 32), v_hi = uint32_t(dv >> 32);
      const uint32_t q_lo = uint32_t(dq), k_lo = uint32_t(dk), p_lo = uint32_t(dp), v_lo = uint32_t(dv);
      auto km_off = [](int kk) { return uint32_t(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4); };   // K-major operand, 64-wide chunks
      auto issue_qk = [&](int j) -> bool {   // S[j & 1] = Q.K_j^T
        const int st = j & 1;
        if (!mbar_wait(k_full + 8u * st, uint32_t(j >> 1) & 1u)) { fail |= 0x20u; return false; }
        tc_fence_after();
        const uint32_t kb = k_lo + uint32_t(st) * (kTile >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          umma_bf16_lohi(tS + uint32_t(st * TK), q_lo + km_off(kk), q_hi, kb + (p.k_mn_major ? uint32_t(kk * 128) : km_off(kk)), k_hi,
                         idesc_s, kk > 0 ? 1u : 0u);
        umma_commit(s_full + 8u * st);
        return true;
      };
      bool ok = mbar_wait(bar_q, 0);
      if (!ok) fail |= 0x10u;
      ok = ok && issue_qk(0);
      if (ok && n_kv > 1) ok = issue_qk(1);
      for (int j = 0; ok && j < n_kv; ++j) {
        const int st = j & 1;
        const uint32_t ph = uint32_t(j >> 1) & 1u;
        // P_j is in shared memory and S tile st has been read
        if (!mbar_wait(p_full + 8u * st, ph)) { fail |= 0x200u; ok = false; break; }
        if (!mbar_wait(v_full + 8u * st, ph)) { fail |= 0x20u; ok = false; break; }
        tc_fence_after();
        const uint32_t vb = v_lo + uint32_t(st) * (kTile >> 4), pb = p_lo + uint32_t(st) * (kPBytes >> 4);
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk)   // O accumulates across key tiles
          umma_bf16_lohi(tO, pb + km_off(kk), p_hi,
                         vb + (p.v_k_major ? uint32_t(((kk >> 2) * (D * 128) + (kk & 3) * 32) >> 4) : uint32_t(kk * 128)), v_hi, idesc_o,
                         (j > 0 || kk > 0) ? 1u : 0u);
        umma_commit(o_done + 8u * st);
        if (j + 2 < n_kv && !issue_qk(j + 2)) { ok = false; break; }   // into the S tile that was just read
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(p.status, 0x100u | fail);
      }
    }
  } else {
    // ======================= softmax (256 threads, two per query row) =======================
    const int row = threadIdx.x & 127, half = threadIdx.x >> 7;
    const int qi = m0 + row;
    const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;   // warps w and w+4 share a lane quarter
    constexpr int HC = TK / 2;
    const int cbase = half * HC;
    // m_used is the (possibly stale) row maximum the exponentials are taken against; O (in tensor
    // memory) and l are rescaled only when the true maximum has moved by more than 2^8, so most
    // key tiles accumulate P.V straight into tensor memory with no traffic on O at all.
    float m_used = -INFINITY, l_run = 0.f;
    bool ok = true;
    uint32_t fail = 0;
    for (int j = 0; j < n_kv; ++j) {
      const int st = j & 1;
      const uint32_t ph = uint32_t(j >> 1) & 1u;
      const int kv0 = j * TK;
      if (ok && !mbar_wait(s_full + 8u * st, ph)) { ok = false; fail |= 0x40u; }
      tc_fence_after();
      // ---- this thread owns half (64 columns) of query row qi: read its scores once ----
      uint32_t r[HC];
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32)
        tmem_ld32(tS + uint32_t(st * TK) + lane_addr + cbase + c0, *reinterpret_cast<uint32_t(*)[32]>(&r[c0]));
      tmem_ld_wait();
      const int kv_lim = (p.causal ? min(p.S, qi + 1) : p.S) - kv0 - cbase;   // local columns >= kv_lim are masked
      const bool full = kv_lim >= HC;
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (full) {
#pragma unroll
        for (int i = 0; i < HC; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
      } else {
#pragma unroll
        for (int i = 0; i < HC; ++i)
          if (i < kv_lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
      }
      float* xj = xch + st * 256;
      xj[half * 128 + row] = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      if (!ok) *abort_flag = 1;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*abort_flag) { ok = false; break; }   // read right after the barrier: every thread sees the same value
      // The reference point of the exponentials is rounded up to a whole number (base-2 domain): every P entry is
      // then 2^(t - n) with n an integer, so its bf16 rounding is that of 2^t itself, the same whichever tile
      // first set the maximum and however often it moved, and the rescale factors below are exact powers of two.
      const float m_tile = ceilf(fmaxf(xj[row], xj[128 + row]) * p.scale_log2);
      if (j == 0) {
        m_used = m_tile;
      } else {
        const bool need = m_tile > m_used + 8.f;
        if (__any_sync(0xffffffffu, need)) {
          // every P.V issued so far must have landed in O before it is rescaled
          if (!mbar_wait(o_done + 8u * ((j - 1) & 1), uint32_t((j - 1) >> 1) & 1u)) { ok = false; fail |= 0x80u; }
          tc_fence_after();
          const float m_new = need ? m_tile : m_used;
          const float alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - m_new);
#pragma unroll 1
          for (int c0 = half * (D / 2); c0 < (half + 1) * (D / 2); c0 += 32) {
            uint32_t q[32];
            tmem_ld32(tO + lane_addr + c0, q);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) q[i] = __float_as_uint(__uint_as_float(q[i]) * alpha);
            tmem_st32(tO + lane_addr + c0, q);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          l_run *= alpha;
          m_used = m_new;
        }
      }
      // P tile st was last read by P_{j-2}.V_{j-2}
      if (j >= 2 && ok && !mbar_wait(o_done + 8u * st, uint32_t((j - 2) >> 1) & 1u)) { ok = false; fail |= 0x80u; }
      // ---- P = exp2(s * k - m_used), bf16, into the swizzled K-major tile (this thread's 64 columns
      //      are exactly one 64-column chunk of the tile) ----
      float ps4[4] = {0.f, 0.f, 0.f, 0.f};
      const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
      uint8_t* p_tile = p_smem + st * kPBytes + half * 16384u + row * 128u;
#pragma unroll
      for (int g = 0; g < HC / 8; ++g) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int col = g * 8 + 2 * i;
          float a = ex2_fast(fmaf(__uint_as_float(r[col]), p.scale_log2, neg_m));
          float bb = ex2_fast(fmaf(__uint_as_float(r[col + 1]), p.scale_log2, neg_m));
          if (!full) {
            if (col >= kv_lim) a = 0.f;
            if (col + 1 >= kv_lim) bb = 0.f;
          }
          const __nv_bfloat162 hv = __floats2bfloat162_rn(a, bb);
          w[i] = *reinterpret_cast<const uint32_t*>(&hv);
          ps4[i] += a + bb;   // fp32 sum; the bf16 rounding of P averages out of the normalisation (relative 2^-9 / sqrt(n))
        }
        *reinterpret_cast<uint4*>(p_tile + ((g ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      l_run += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);   // partial sum over this thread's columns
      // generic-proxy writes of P -> visible to the tensor core; this thread is done with S tile st
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      mbar_arrive(p_full + 8u * st);
    }
    // ---- O / l -> bf16 ----
    if (ok && n_kv > 0) {
      if (!mbar_wait(o_done + 8u * ((n_kv - 1) & 1), uint32_t((n_kv - 1) >> 1) & 1u)) { ok = false; fail |= 0x80u; }
      tc_fence_after();
    }
    if (fail) atomicOr(p.status, 0x100u | fail);
    if (!ok) *abort_flag = 1;
    float* xl = xch + (n_kv & 1) * 256;   // the exchange buffer the last tile did not use
    xl[half * 128 + row] = l_run;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (!*abort_flag) {
      const float l_tot = xl[row] + xl[128 + row];
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.O) + (int64_t)b * p.o_s[0] + (int64_t)h * p.o_s[1] + (int64_t)qi * p.o_s[2];
      pdl_wait();  // O may still be read by an earlier step
#pragma unroll 1
      for (int c0 = half * (D / 2); c0 < (half + 1) * (D / 2); c0 += 32) {
        uint32_t q[32];
        tmem_ld32(tO + lane_addr + c0, q);     // warp-collective: rows past the end take part, then skip the store
        tmem_ld_wait();
        if (qi < p.S) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(q[g * 8 + i]) * inv;
            store16(out + c0 + g * 8, v);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}


// ---- two query tiles per work item, probabilities in tensor memory ----------------------------------------------
// A work item = one (batch, head) and 256 consecutive queries, as two 128-row tiles ("slots") that share every K / V
// tile loaded for the item. Warps 0-3 are the softmax of slot 0, warps 4-7 of slot 1 (one thread per query row: the
// row's maximum and sum never leave the thread), warp 8 issues every tcgen05.mma, warp 9 the TMA loads. Tensor memory:
// S_0, S_1 (128 fp32 columns each), O_0, O_1 (D columns each). A softmax thread reads its row of S_t, writes the bf16
// probabilities back over the same columns (two per 32-bit column, 64 columns), and P_t.V runs with the A operand
// taken from tensor memory: P never passes through shared memory. Per slot the chain S = Q.K_j^T -> softmax ->
// O += P.V_j is serial; the two slots run half a step apart, so the tensor core works for one while the other's
// softmax runs.
//   q_full        both Q tiles of the item have landed                TMA -> MMA
//   q_free        the item's last Q.K^T has read them                 MMA commit -> loader
//   k_full[s], v_full[s]   K / V stage s has landed                   TMA -> MMA
//   k_free[s], v_free[s]   every MMA that reads stage s is complete   MMA commit -> loader
//   s_full[t]     S_t holds Q_t.K_j^T                                 MMA commit -> softmax t
//   p_full[t]     P_t is written (and S_t read)                       128 softmax threads -> MMA
//   o_done[t]     O_t holds P_t.V_j                                   MMA commit -> softmax t (rescale, end)
//   o_free[t]     the item's output has been read out of O_t          128 softmax threads -> MMA
// What sets the pace (clock stamps in both roles, non-causal 2 x 4096 x 32 x 128): a slot's step is softmax ~2000
// cycles (maximum pass 450, exponential pass 1530: 128 exponentials per thread at 4 per clock and scheduler), then
// ~1900 cycles in which the MMA warp takes its three waits (~450) and issues the 8 + 8 instructions of P.V and the next
// Q.K^T (~700 + ~750, i.e. ~90 cycles an instruction against 64 alone). The MMA warp serves the two slots in turn and
// is busy throughout, so a step of both slots takes ~4050 cycles for 2 x 1024 cycles of tensor-core work. The ~90
// cycles are the tensor core's own pace here, not the issuing warp's: with every product's instructions split between
// two issuing warps on two schedulers (which in a probe brings 110 cycles per instruction beside arithmetic warps back
// to 64) the kernel ran exactly as fast (951 vs 954 TFLOP/s); and with one issuing warp per slot the slots fall into
// step, their softmax passes share the schedulers and their products the pipe (757 TFLOP/s).
// Forms for a role that the whole warp runs in lockstep: every lane executes the instruction, one lane's carries a true
// issue predicate.
__device__ __forceinline__ void umma_ss_elect(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc,
                                              uint32_t leader) {
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.b32 p, %4, 0;\n setp.ne.b32 q, %5, 0;\n"
      " @q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(leader) : "memory");
}
__device__ __forceinline__ void umma_ts_elect(uint32_t tmem_c, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc,
                                              uint32_t leader) {
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.b32 p, %4, 0;\n setp.ne.b32 q, %5, 0;\n"
      " @q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      ::"r"(tmem_c), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc), "r"(leader) : "memory");
}
// Every MMA of one product (Q.K^T over the head dim, P.V over a key tile) in ONE asm block: the predicates are set once
// and the descriptors advance by immediates, so an instruction costs the issuing warp two additions and itself. The
// warp shares its scheduler with softmax warps, and every instruction it does not issue leaves the tensor cores
// waiting less (measured alone: 64 cycles per 128 x 128 x 16 instruction either way; beside two warps issuing
// fused multiply-adds on the same scheduler: 115 per instruction one by one, 108 in blocks, 186 when those warps
// issue nothing else; special-function and integer instructions beside it cost nothing).
#define FLUID_MMA_SS_1(OA, OB) \
    " add.s64 a, %1, " #OA "; add.s64 b, %2, " #OB ";\n @q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, one;\n"
#define FLUID_MMA_SS_HEAD \
    "{\n .reg .pred q, one;\n .reg .b64 a, b;\n setp.ne.b32 q, %4, 0;\n setp.eq.b32 one, 0, 0;\n" \
    " @q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, !one;\n"
#define FLUID_MMA_SS_ARGS ::"r"(tmem_c), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(leader) : "memory"
// S = Q.K^T: the first instruction overwrites the accumulator. kk-th offsets: A K-major in 64-wide chunks; B likewise,
// or MN-major (128 descriptor units per 16 keys).
template <int D, bool B_MN>
__device__ __forceinline__ void umma_qk_block(uint32_t tmem_c, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t leader) {
  if (D == 64) {
    if (!B_MN) asm volatile(FLUID_MMA_SS_HEAD FLUID_MMA_SS_1(2, 2) FLUID_MMA_SS_1(4, 4) FLUID_MMA_SS_1(6, 6) "}" FLUID_MMA_SS_ARGS);
    else asm volatile(FLUID_MMA_SS_HEAD FLUID_MMA_SS_1(2, 128) FLUID_MMA_SS_1(4, 256) FLUID_MMA_SS_1(6, 384) "}" FLUID_MMA_SS_ARGS);
  } else {
    if (!B_MN) asm volatile(FLUID_MMA_SS_HEAD FLUID_MMA_SS_1(2, 2) FLUID_MMA_SS_1(4, 4) FLUID_MMA_SS_1(6, 6) FLUID_MMA_SS_1(1024, 1024)
                            FLUID_MMA_SS_1(1026, 1026) FLUID_MMA_SS_1(1028, 1028) FLUID_MMA_SS_1(1030, 1030) "}" FLUID_MMA_SS_ARGS);
    else asm volatile(FLUID_MMA_SS_HEAD FLUID_MMA_SS_1(2, 128) FLUID_MMA_SS_1(4, 256) FLUID_MMA_SS_1(6, 384) FLUID_MMA_SS_1(1024, 512)
                      FLUID_MMA_SS_1(1026, 640) FLUID_MMA_SS_1(1028, 768) FLUID_MMA_SS_1(1030, 896) "}" FLUID_MMA_SS_ARGS);
  }
}
#define FLUID_MMA_TS_1(OA, OB) \
    " add.u32 a, %1, " #OA "; add.s64 b, %2, " #OB ";\n @q tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, one;\n"
#define FLUID_MMA_TS_HEAD \
    "{\n .reg .pred p, q, one;\n .reg .b64 b;\n .reg .b32 a;\n setp.ne.b32 p, %4, 0;\n setp.ne.b32 q, %5, 0;\n setp.eq.b32 one, 0, 0;\n" \
    " @q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
#define FLUID_MMA_TS_ARGS ::"r"(tmem_c), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc), "r"(leader) : "memory"
// O (+)= P.V over one 128-key tile: eight instructions of 16 keys (8 packed columns of P each); acc: whether the first
// one adds to O. B offsets: V with d contiguous (MN-major: 128 units per 16 keys) or with keys contiguous (K-major in
// 64-key chunks of D rows).
template <int D, bool V_K>
__device__ __forceinline__ void umma_pv_block(uint32_t tmem_c, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc, uint32_t leader) {
  if (!V_K)
    asm volatile(FLUID_MMA_TS_HEAD FLUID_MMA_TS_1(8, 128) FLUID_MMA_TS_1(16, 256) FLUID_MMA_TS_1(24, 384) FLUID_MMA_TS_1(32, 512)
                 FLUID_MMA_TS_1(40, 640) FLUID_MMA_TS_1(48, 768) FLUID_MMA_TS_1(56, 896) "}" FLUID_MMA_TS_ARGS);
  else if (D == 64)
    asm volatile(FLUID_MMA_TS_HEAD FLUID_MMA_TS_1(8, 2) FLUID_MMA_TS_1(16, 4) FLUID_MMA_TS_1(24, 6) FLUID_MMA_TS_1(32, 512)
                 FLUID_MMA_TS_1(40, 514) FLUID_MMA_TS_1(48, 516) FLUID_MMA_TS_1(56, 518) "}" FLUID_MMA_TS_ARGS);
  else
    asm volatile(FLUID_MMA_TS_HEAD FLUID_MMA_TS_1(8, 2) FLUID_MMA_TS_1(16, 4) FLUID_MMA_TS_1(24, 6) FLUID_MMA_TS_1(32, 1024)
                 FLUID_MMA_TS_1(40, 1026) FLUID_MMA_TS_1(48, 1028) FLUID_MMA_TS_1(56, 1030) "}" FLUID_MMA_TS_ARGS);
}
__device__ __forceinline__ void umma_commit_elect(uint32_t bar, uint32_t leader) {
  asm volatile(
      "{\n .reg .pred q;\n setp.ne.b32 q, %1, 0;\n"
      " @q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}"
      ::"r"(bar), "r"(leader) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&q)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]), "r"(q[4]), "r"(q[5]), "r"(q[6]), "r"(q[7]), "r"(q[8]),
      "r"(q[9]), "r"(q[10]), "r"(q[11]), "r"(q[12]), "r"(q[13]), "r"(q[14]), "r"(q[15])
      : "memory");
}
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// two fp32 lanes in one 64-bit register: one issue slot for two fused multiply-adds / additions
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for x <= 0 on the fused-multiply-add pipe (no special-function unit): nearest-integer split by the 1.5 * 2^23
// trick, degree-4 polynomial for 2^f on [-0.5, 0.5] (relative error < 3e-6, far below the bf16 rounding of P), the
// integer part added into the exponent field. A share of each tile's exponentials goes this way so that the
// special-function unit (4 lanes per clock and scheduler) is not what a softmax warp waits for.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -125.f);
  const float z = x + 12582912.f;
  const float f = x - (z - 12582912.f);
  float q = fmaf(0.009582852944731712f, f, 0.055906426161527634f);
  q = fmaf(q, f, 0.24024099111557007f);
  q = fmaf(q, f, 0.6931241750717163f);
  q = fmaf(q, f, 1.0f);
  return __int_as_float(__float_as_int(q) + (__float_as_int(z) << 23));
}

// Two query tiles per CTA, persistent: gridDim.x CTAs (one per SM) walk the launch's work items. A work item is a pair
// of adjacent 128-row query tiles of one (batch, head); items are numbered heaviest first (with a causal mask the last
// query tiles see the most key tiles) and dealt to the CTAs in a snake (round r: CTA c takes item r P + c when r is
// even, r P + P - 1 - c when odd), which for weights that fall with the item number is the longest-first rule: the
// CTA that drew the heaviest item of a round draws the lightest of the next. Nothing is torn down between items:
// tensor memory and barriers stay, the key / value ring keeps running across the boundary, the next item's query
// tiles are fetched as soon as the last Q.K^T of the current one has read them, and its first scores are computed
// while the softmax warps still normalise and store the current output. (As one CTA per item, a second CTA on an SM
// started 3.7 us after the first had left and spent another 3 us before its first instruction on the tensor cores;
// the causal Llama-shaped launch of 256 items took 49.6 us for 39.4 us of its heaviest item.)
// Barrier phases count completions over the whole launch, not per item: kc key / value tiles loaded before this item,
// sc[t] score tiles of slot t, oc[t] items in which slot t was active.
template <int D>
__global__ void __launch_bounds__(320, 1)
attn_tc2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ AttnParams p) {
  constexpr int DC = D / 64;                       // 64-wide chunks of the head dim
  constexpr uint32_t kTile = TQ * D * 2;           // bytes of one Q / K / V tile
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sQ = raw, sK = sQ + 2 * kTile, sV = sK + 2 * kTile, bars = sV + 2 * kTile;
  const uint32_t q_full = bars, k_full = bars + 8, v_full = bars + 24, k_free = bars + 40, v_free = bars + 56,
                 s_full = bars + 72, p_full = bars + 88, o_done = bars + 104, q_free = bars + 120, o_free = bars + 128;
  const uint32_t tmem_slot = bars + 144;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  volatile uint32_t* abort_flag = tmem_slot_ptr + 1;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_bz = p.B * p.NH;
  const int n_mt = (p.S + 2 * TQ - 1) / (2 * TQ);
  const int n_items = n_mt * n_bz;
  const int n_cta = int(gridDim.x), cta = int(blockIdx.x);
  // r-th item of this CTA, -1 past the end (a CTA without an item in round r has none in a later round either)
  auto item_of = [&](int r) -> int {
    const int idx = r * n_cta + ((r & 1) ? n_cta - 1 - cta : cta);
    return idx < n_items ? idx : -1;
  };
  struct Item { int bz, m0, n_kv[2], n_max; };
  auto decode = [&](int it, Item& w) {
    w.bz = it % n_bz;
    w.m0 = ((n_mt - 1) - it / n_bz) * 2 * TQ;
    // key tiles each query tile needs (0: the tile lies beyond the sequence)
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int mq = w.m0 + t * TQ;
      int n = mq < p.S ? (p.S + TK - 1) / TK : 0;
      if (p.causal && n) n = min(n, (mq + TQ - 1) / TK + 1);
      w.n_kv[t] = n;
    }
    w.n_max = max(w.n_kv[0], w.n_kv[1]);
  };
  if (raw & 1023u) {   // cannot happen with the launch this file does; refuse rather than run misaligned tiles
    if (threadIdx.x == 0) atomicOr(p.status, 0x100u | 0x08u);
    return;
  }

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_free, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(k_full + 8 * i, 1); mbar_init(v_full + 8 * i, 1); mbar_init(k_free + 8 * i, 1); mbar_init(v_free + 8 * i, 1);
      mbar_init(s_full + 8 * i, 1); mbar_init(p_full + 8 * i, 128); mbar_init(o_done + 8 * i, 1); mbar_init(o_free + 8 * i, 128);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  // S_t at columns 128 t (P_t over its first 64), O_t at 256 + D t

  constexpr int kMmaWarp = 8, kLoadWarp = 9;
  if (warp == kLoadWarp) {
    // ======================= loads =======================
    const bool lead = lane == 0;
    constexpr int NB = 2 * DC;               // boxes per tile
    const bool k_lane = lane < NB, v_lane = lane >= NB && lane < 2 * NB;
    const int bx = k_lane ? lane : lane - NB;
    int cur[5] = {0, 0, 0, 0, 0}, inc[5] = {0, 0, 0, 0, 0};
    uint32_t box_dst = 0;
    // this lane's box of a K / V tile: where it lands, and its coordinates at key tile 0 of (batch, head) bz
    auto start_head = [&](int bz) {
      if (k_lane) {
        if (!p.k_mn_major) {          // [d chunk][128 keys][64 d]: box (dc, rh)
          const int dc = bx >> 1, rh = bx & 1;
          coords(p.k_sel, dc * 64, rh * 64, bz, p.k_b0, cur);
          box_dst = sK + dc * 16384u + rh * 8192u;
        } else {                      // [key chunk][D d-rows][64 keys]: box (sc, dc)
          const int sc = bx / DC, dc = bx % DC;
          coords(p.k_sel, dc * 64, sc * 64, bz, p.k_b0, cur);
          box_dst = sK + sc * (D * 128u) + dc * 8192u;
        }
      } else if (v_lane) {
        if (!p.v_k_major) {           // [d chunk][128 keys][64 d]  (MN-major B of P.V): box (dc, kc)
          const int dc = bx >> 1, kc = bx & 1;
          coords(p.v_sel, kc * 64, dc * 64, bz, p.v_b0, cur);
          box_dst = sV + dc * 16384u + kc * 8192u;
        } else {                      // [key chunk][D d-rows][64 keys]  (K-major B of P.V): box (kc, dh)
          const int kc = bx / DC, dh = bx % DC;
          coords(p.v_sel, kc * 64, dh * 64, bz, p.v_b0, cur);
          box_dst = sV + kc * (D * 128u) + dh * 8192u;
        }
      }
    };
    if (k_lane) {
#pragma unroll
      for (int d = 0; d < 5; ++d) inc[d] = p.k_sel[d] == 2 ? TK : 0;
    } else if (v_lane) {
#pragma unroll
      for (int d = 0; d < 5; ++d) inc[d] = p.v_sel[d] == 0 ? TK : 0;
    }
    uint32_t fail = 0;
    int kc = 0;         // key / value tiles issued so far, over all items: tile kc lands in stage kc & 1
    int q_issued = 0;   // items whose query tiles have been issued
    auto load_kv = [&](bool is_k) {
      const uint32_t bar = (is_k ? k_full : v_full) + 8u * (kc & 1);
      if (lead) mbar_expect_tx(bar, kTile);
      if (is_k ? k_lane : v_lane) {
        tma_load5(box_dst + uint32_t(kc & 1) * kTile, is_k ? &map_k : &map_v, bar, cur);
#pragma unroll
        for (int d = 0; d < 5; ++d) cur[d] += inc[d];
      }
    };
    auto all_ok = [&](bool mine) { return __shfl_sync(0xffffffffu, mine ? 1 : 0, 0) != 0; };   // lane 0 decides

    bool ok = true;
    for (int r = 0; ok; ++r) {
      const int it = item_of(r);
      if (it < 0) break;
      Item w;
      decode(it, w);
      start_head(w.bz);
      if (r == 0) pdl_wait();  // Q, K, V come from the previous steps (the first item's coordinates above do not)
      if (r > 0) {   // the previous item's last Q.K^T has read the query tiles
        if (lead && !mbar_wait(q_free, uint32_t(r - 1) & 1u)) { fail |= 0x10u; ok = false; }
        ok = all_ok(ok && !*abort_flag);
        if (!ok) break;
      }
      if (lead) {
        const int n_q = w.n_kv[1] ? 2 : 1;
        mbar_expect_tx(q_full, uint32_t(n_q) * kTile);
        int c[5];
        for (int t = 0; t < n_q; ++t)
          for (int dc = 0; dc < DC; ++dc)
            for (int rh = 0; rh < 2; ++rh) {
              coords(p.q_sel, dc * 64, w.m0 + t * TQ + rh * 64, w.bz, p.q_b0, c);
              tma_load5(sQ + uint32_t(t) * kTile + dc * 16384u + rh * 8192u, &map_q, q_full, c);
            }
      }
      q_issued = r + 1;
      for (int j = 0; j < w.n_max; ++j) {
        // stage kc & 1 is free once the tile loaded two before (kc - 2) has been read: completion (kc - 2) / 2 of its barrier
        const uint32_t ph = uint32_t((kc - 2) >> 1) & 1u;
        if (kc >= 2) {
          if (lead && !mbar_wait(k_free + 8u * (kc & 1), ph)) { fail |= 0x40u; ok = false; }
          ok = all_ok(ok);
          if (!ok) break;
        }
        load_kv(true);
        if (kc >= 2) {
          if (lead && !mbar_wait(v_free + 8u * (kc & 1), ph)) { fail |= 0x80u; ok = false; }
          ok = all_ok(ok && !*abort_flag);
          if (!ok) {   // the K tile of this index is in flight, its V tile is not
            if (lead) mbar_wait(k_full + 8u * (kc & 1), uint32_t(kc >> 1) & 1u);
            break;
          }
        }
        load_kv(false);
        ++kc;
      }
    }
    if (!ok && lead) {
      *abort_flag = 1;
      if (fail) atomicOr(p.status, 0x100u | fail);
    }
    if (lead && *abort_flag) {
      // let loads still in flight land before the shared memory is given up (each wait is bounded)
      if (q_issued > 0) mbar_wait(q_full, uint32_t(q_issued - 1) & 1u);
      for (int j = max(0, kc - 2); j < kc; ++j) {
        mbar_wait(k_full + 8u * (j & 1), uint32_t(j >> 1) & 1u);
        mbar_wait(v_full + 8u * (j & 1), uint32_t(j >> 1) & 1u);
      }
    }
  } else if (warp == kMmaWarp) {
    // ======================= MMAs =======================
    // The whole warp runs this role in lockstep and one lane's instructions carry the issue predicate. A probe with this
    // very issue code and nothing else on the SM runs a 128 x 128 x 16 instruction every 64 cycles (convergent or under
    // a one-lane branch alike, also with eight warps reading and writing tensor memory beside it: 66). What slows it is
    // arithmetic on the SAME scheduler: beside two warps there that issue fused multiply-adds back to back an
    // instruction takes 115-186 cycles, beside warps that issue only special-function or integer instructions, or that
    // sit on the other three schedulers, 64-77. Every scheduler carries one softmax warp of each slot (a warp reaches
    // only the tensor-memory lanes of its own quarter), so this role cannot be moved out of their way. It does not have
    // to be: two issuing warps (each half of every product, handed over through a named barrier and the tensor-core
    // fences) left the kernel's time unchanged, so in the kernel the issue is not what the tensor core waits for.
    {
      const uint32_t leader = lane == 0 ? 1u : 0u;
      uint32_t fail = 0;
      const uint32_t idesc_s = make_idesc(TK, 0, p.k_mn_major);
      const uint32_t idesc_o = make_idesc(D, 0, p.v_k_major ? 0 : 1);
      const uint64_t dq = make_desc(sQ, 16, 1024);
      const uint64_t dk = p.k_mn_major ? make_desc(sK, D * 128u, 1024) : make_desc(sK, 16, 1024);
      const uint64_t dv = p.v_k_major ? make_desc(sV, 16, 1024) : make_desc(sV, 16384, 1024);
      auto km_off = [](int kk) { return uint64_t(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4); };   // K-major operand, 64-wide chunks
      const uint32_t tm = __shfl_sync(0xffffffffu, tmem_base, 0);
      Item w;
      int kc0 = 0;              // key / value tiles of the items before this one
      int sc[2] = {0, 0};       // score tiles of slot t before this item (= softmax passes = P.V products)
      int oc[2] = {0, 0};       // items before this one in which slot t was active
      int last_t = 0, qk_left = 0;
      auto issue_qk = [&](int t, int j) -> bool {   // S_t = Q_t.K_j^T
        const int kc = kc0 + j, st = kc & 1;
        if (!mbar_wait_warp(k_full + 8u * st, uint32_t(kc >> 1) & 1u)) { fail |= 0x20u; return false; }
        tc_fence_after();
        const uint64_t kb = dk + uint64_t(st) * (kTile >> 4), qb = dq + uint64_t(t) * (kTile >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          umma_ss_elect(tm + uint32_t(t * TK), qb + km_off(kk), kb + (p.k_mn_major ? uint64_t(kk * 128) : km_off(kk)), idesc_s,
                        kk > 0 ? 1u : 0u, leader);
        umma_commit_elect(s_full + 8u * t, leader);
        if (t == last_t || j >= w.n_kv[1]) umma_commit_elect(k_free + 8u * st, leader);
        if (--qk_left == 0) umma_commit_elect(q_free, leader);   // the item's query tiles have been read for the last time
        return true;
      };
      auto issue_pv = [&](int t, int j) -> bool {   // O_t += P_t.V_j
        const int kc = kc0 + j, st = kc & 1;
        // the first product of an item overwrites O_t: the previous item's output must have been read out of it
        if (j == 0 && oc[t] > 0 && !mbar_wait_warp(o_free + 8u * t, uint32_t(oc[t] - 1) & 1u)) { fail |= 0x400u; return false; }
        if (!mbar_wait_warp(p_full + 8u * t, uint32_t(sc[t] + j) & 1u)) { fail |= 0x200u; return false; }
        if (!mbar_wait_warp(v_full + 8u * st, uint32_t(kc >> 1) & 1u)) { fail |= 0x20u; return false; }
        tc_fence_after();
        const uint64_t vb = dv + uint64_t(st) * (kTile >> 4);
        const uint32_t tP = tm + uint32_t(t * TK), tO = tm + 2 * TK + uint32_t(t * D);
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk)   // 16 keys = 8 packed columns of P per instruction
          umma_ts_elect(tO, tP + uint32_t(kk * 8),
                        vb + (p.v_k_major ? uint64_t(((kk >> 2) * (D * 128) + (kk & 3) * 32) >> 4) : uint64_t(kk * 128)), idesc_o,
                        (j > 0 || kk > 0) ? 1u : 0u, leader);
        umma_commit_elect(o_done + 8u * t, leader);
        if (t == last_t || j >= w.n_kv[1]) umma_commit_elect(v_free + 8u * st, leader);
        return true;
      };
      bool ok = true;
      for (int r = 0; ok; ++r) {
        const int it = item_of(r);
        if (it < 0) break;
        decode(it, w);
        last_t = w.n_kv[1] ? 1 : 0;    // the tile whose MMA is the last reader of a K / V stage (n_kv[1] >= n_kv[0] when tile 1 exists)
        qk_left = w.n_kv[0] + w.n_kv[1];
        ok = mbar_wait_warp(q_full, uint32_t(r) & 1u);
        if (!ok) fail |= 0x10u;
        for (int t = 0; ok && t < 2; ++t)
          if (w.n_kv[t] > 0) ok = issue_qk(t, 0);
        for (int j = 0; ok && j < w.n_max; ++j) {
          for (int t = 0; ok && t < 2; ++t) {
            if (j >= w.n_kv[t]) continue;
            ok = issue_pv(t, j);
            if (ok && j + 1 < w.n_kv[t]) ok = issue_qk(t, j + 1);   // into the S tile whose probabilities were just consumed
          }
        }
        kc0 += w.n_max;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          sc[t] += w.n_kv[t];
          oc[t] += w.n_kv[t] > 0 ? 1 : 0;
        }
      }
      if (!ok && leader) {
        *abort_flag = 1;
        atomicOr(p.status, 0x100u | fail);
      }
    }
  } else {
    // ======================= softmax: warps 0-3 query tile 0, warps 4-7 query tile 1 =======================
    const int t = warp >> 2, row = threadIdx.x & 127;
    const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + lane_addr + uint32_t(t * TK);
    const uint32_t tO = tmem_base + lane_addr + 2 * TK + uint32_t(t * D);
    bool ok = true;
    uint32_t fail = 0;
    int sc = 0;   // score tiles of this slot before the current item
    // (Making the two softmax groups take turns through a pair of named barriers, so that they never share the
    // schedulers, was measured and is slower: 918 -> 876 TFLOP/s on 2 x 4096 x 32 x 128. A pass is bound by what one
    // warp can issue alone, so two groups running together get more out of a scheduler than one at a time. Two threads
    // per row (twice the warps) was measured no faster either, 940 vs 958 TFLOP/s: the tensor side sets the pace.)
    for (int r = 0; ok; ++r) {
      const int it = item_of(r);
      if (it < 0) break;
      Item w;
      decode(it, w);
      const int n = w.n_kv[t];
      const int qi = w.m0 + t * TQ + row;
      float m_used = -INFINITY, l_run = 0.f;
      for (int j = 0; j < n; ++j) {
        if (!mbar_wait_warp(s_full + 8u * t, uint32_t(sc + j) & 1u)) { ok = false; fail |= 0x40u; break; }
        const int kv0 = j * TK;
        tc_fence_after();
        // Two passes over the row of S, 32 columns at a time, so that a thread holds 64 scores at most (with all 128 in
        // registers the kernel spills at the 168 registers ten warps leave a thread). Pass 1: the row maximum.
        const int kv_lim = (p.causal ? min(p.S, qi + 1) : p.S) - kv0;   // local columns >= kv_lim are masked
        // one answer per warp: both branches of pass 2 issue warp-collective tensor-memory stores (on the diagonal
        // tile the last row of a warp sees every column while the other rows do not)
        const bool full = __all_sync(0xffffffffu, kv_lim >= TK);
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        {
          uint32_t q[2][32];
          tmem_ld32(tS, q[0]);
#pragma unroll
          for (int c = 0; c < TK / 32; ++c) {
            tmem_ld_wait();
            if (c + 1 < TK / 32) tmem_ld32(tS + (c + 1) * 32, q[(c + 1) & 1]);
            if (full) {
#pragma unroll
              for (int i = 0; i < 32; i += 8)
#pragma unroll
                for (int u = 0; u < 4; ++u)
                  mx4[u] = max3(mx4[u], __uint_as_float(q[c & 1][i + 2 * u]), __uint_as_float(q[c & 1][i + 2 * u + 1]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c * 32 + i < kv_lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(q[c & 1][i]));
            }
          }
        }
        // whole-number reference point (base-2 domain): P's bf16 rounding is then that of 2^t itself and the rescale
        // factors are exact powers of two
        const float m_tile = ceilf(fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2);
        if (j == 0) {
          m_used = m_tile;
        } else {
          const bool need = m_tile > m_used + 8.f;
          if (__any_sync(0xffffffffu, need)) {
            // P_{j-1}.V_{j-1} must have landed in O before it is rescaled
            if (!mbar_wait_warp(o_done + 8u * t, uint32_t(sc + j - 1) & 1u)) { ok = false; fail |= 0x80u; break; }
            tc_fence_after();
            const float m_new = need ? m_tile : m_used;
            const float alpha = exp2f(m_used - m_new);
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 32) {
              uint32_t q[32];
              tmem_ld32(tO + c0, q);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) q[i] = __float_as_uint(__uint_as_float(q[i]) * alpha);
              tmem_st32(tO + c0, q);
            }
            l_run *= alpha;
            m_used = m_new;
          }
        }
        // Pass 2: P = exp2(s * k - m_used) as bf16 pairs over S's first 64 columns. Chunk c (columns 32c..32c+31) is
        // read before P chunk c (packed columns 16c..16c+15) is written, and the chunk read ahead lies above both.
        float ps4[4] = {0.f, 0.f, 0.f, 0.f};
        const float neg_m = -m_used;
        {
          const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(neg_m, neg_m);
          uint64_t acc[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
          uint32_t q[2][32];
          tmem_ld32(tS, q[0]);
#pragma unroll
          for (int c = 0; c < TK / 32; ++c) {
            tmem_ld_wait();
            if (c + 1 < TK / 32) tmem_ld32(tS + (c + 1) * 32, q[(c + 1) & 1]);
            uint32_t wv[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float x0, x1;
              unpack2(fma2(pack2(__uint_as_float(q[c & 1][2 * i]), __uint_as_float(q[c & 1][2 * i + 1])), sc2, nm2), x0, x1);
              float a, bb;
              if (kPolyEvery > 0 && (i % (kPolyEvery > 0 ? kPolyEvery : 1)) == 0) { a = ex2_poly(x0); bb = ex2_poly(x1); }
              else { a = ex2_fast(x0); bb = ex2_fast(x1); }
              if (!full) {
                if (c * 32 + 2 * i >= kv_lim) a = 0.f;
                if (c * 32 + 2 * i + 1 >= kv_lim) bb = 0.f;
              }
              wv[i] = pack_bf16x2(a, bb);
              acc[i & 1] = add2(acc[i & 1], pack2(a, bb));   // fp32 sum of the unrounded exponentials
            }
            tmem_st16(tS + c * 16, wv);
          }
          unpack2(acc[0], ps4[0], ps4[1]);
          unpack2(acc[1], ps4[2], ps4[3]);
        }
        l_run += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        mbar_arrive(p_full + 8u * t);
      }
      if (!ok) break;
      // ---- O / l -> bf16 ----
      if (n > 0) {
        if (!mbar_wait_warp(o_done + 8u * t, uint32_t(sc + n - 1) & 1u)) { ok = false; fail |= 0x80u; break; }
        tc_fence_after();
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
        const int h = w.bz % p.NH, b = w.bz / p.NH;
        __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.O) + (int64_t)b * p.o_s[0] + (int64_t)h * p.o_s[1] + (int64_t)qi * p.o_s[2];
        pdl_wait();  // O may still be read by an earlier step
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t q[32];
          tmem_ld32(tO + c0, q);     // warp-collective: rows past the end take part, then skip the store
          tmem_ld_wait();
          if (qi < p.S) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              float v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(q[g * 8 + i]) * inv;
              store16(out + c0 + g * 8, v);
            }
          }
        }
        // O_t has been read out: the next item's first P.V may overwrite it
        tc_fence_before();
        mbar_arrive(o_free + 8u * t);
      }
      sc += n;
    }
    if (fail && lane == 0) atomicOr(p.status, 0x100u | fail);
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace

// Which form runs: two query tiles per work item on persistent CTAs (probabilities in tensor memory) when the sequence
// has more than one query tile; for one tile the register form of attn_small.cu when Q, K and V have d contiguous, else
// the one-tile form. FLUID_ATTN_FORM in the environment forces a form (A/B timing): 1 one tile per CTA, 2 the
// persistent two-tile form. FLUID_ATTN_CTAS caps the persistent form's grid (default: one CTA
// per SM).
static int attn_form(const AttnParams& p) {
  static const int forced = [] {
    const char* e = std::getenv("FLUID_ATTN_FORM");
    return e ? std::atoi(e) : 0;
  }();
  if (forced >= 1 && forced <= 2) return forced;
  if (p.S <= TQ && attn_small_eligible(p)) return 3;
  return p.S > TQ ? 2 : 1;
}

static int attn_ctas() {
  static const int n = [] {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const char* e = std::getenv("FLUID_ATTN_CTAS");
    const int cap = e ? std::atoi(e) : 0;
    return cap > 0 ? cap : sms;
  }();
  return n;
}

template <typename K>
static cudaError_t launch_attn_form(K kernel, bool* attr_done, size_t smem, dim3 grid, int threads, cudaStream_t stream,
                                    const CUtensorMap* mq, const CUtensorMap* mk, const CUtensorMap* mv, const AttnParams& p) {
  if (!*attr_done) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    *attr_done = true;
  }
  return launch_k(kernel, grid, threads, smem, stream, *mq, *mk, *mv, p);
}

cudaError_t launch_attn_tc(const AttnParams& p, const AttnHost& host, cudaStream_t stream) {
  const int D = p.D;
  const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(&host.map_q);
  const CUtensorMap* mk = reinterpret_cast<const CUtensorMap*>(&host.map_k);
  const CUtensorMap* mv = reinterpret_cast<const CUtensorMap*>(&host.map_v);
  static bool attr[4] = {false, false, false, false};
  if (D != 64 && D != 128) return cudaErrorInvalidValue;
  const int form = attn_form(p);
  if (form == 3) return launch_attn_small(p, &host, stream);
  if (form == 2) {
    const size_t smem = size_t(6) * TQ * D * 2 + 256 + 1024;
    const int items = ((p.S + 2 * TQ - 1) / (2 * TQ)) * p.B * p.NH;
    const dim3 grid(std::min(items, attn_ctas()));
    return D == 64 ? launch_attn_form(attn_tc2_kernel<64>, &attr[2], smem, grid, 320, stream, mq, mk, mv, p)
                   : launch_attn_form(attn_tc2_kernel<128>, &attr[3], smem, grid, 320, stream, mq, mk, mv, p);
  }
  const size_t smem = size_t(5) * TQ * D * 2 + size_t(2) * TQ * TK * 2 + 128 + 2048;
  const dim3 grid(((p.S + TQ - 1) / TQ) * p.B * p.NH);
  return D == 64 ? launch_attn_form(attn_tc_kernel<64>, &attr[0], smem, grid, kAttnThreads, stream, mq, mk, mv, p)
                 : launch_attn_form(attn_tc_kernel<128>, &attr[1], smem, grid, kAttnThreads, stream, mq, mk, mv, p);
}

}  // namespace fluid
