// Fused attention for short sequences (S <= 128; bf16, head dim 64 or 128, d contiguous in Q, K and V):
// softmax(scale * Q.K^T [+ causal mask]).V for one (batch, head) and 16 query rows per CTA, scores and probabilities
// never in global memory.
//
// Why a second form beside the tcgen05 kernels: at S <= 128 a launch is one key tile per (batch, head), so the
// tensor-memory form runs as a handful of CTAs (12 for a 12-head encoder at batch 1), each a serial chain of TMA
// load -> tcgen05 Q.K^T -> tensor-memory round trip -> softmax -> shared-memory round trip -> tcgen05 P.V -> tensor-memory
// round trip -> store, behind a 512-column tensor-memory allocation and ten barriers. Here the work is cut as finely
// as warp-level mma.sync m16n8k16 allows and spread over many SMs: a CTA owns 16 query rows, its four warps split
// the KEYS for Q.K^T (a quarter of the scores each, in registers), meet once to agree on the row maxima, exchange the
// bf16 probabilities through 4 KB of shared memory, and split the HEAD DIM for P.V (a quarter of the output columns
// each, so no partial outputs are added up). A warp-level MMA takes ~60 cycles here from issue to issue, so a warp
// that ran all 128 of a 16-row block alone took 4.4 us; four warps run 32 each (eight warps with 16 each measured
// slower: 0.483 against 0.477 ms for a twelve-layer encoder step). Q and K arrive first, V behind them, landing under
// Q.K^T and the softmax: as bulk-tensor boxes where the step has tensor maps, else as per-thread cp.async into padded
// rows. The tensor cores are only the arithmetic unit.
// Same numeric reading as the other forms: the reference point of the exponentials is the row maximum rounded up to a
// whole number in the base-2 domain, P is rounded to bf16 for the second product, the row sum uses the unrounded
// exponentials, masked entries are exactly zero.
#include <cuda.h>

#include "device_utils.cuh"

namespace fluid {
namespace {

constexpr int kWarps = 4, kRowsPerCta = 16, kMaxS = 128;
constexpr int kPPitch = kMaxS * 2 + 16;   // bytes per row of the probability tile
constexpr int kKeysPerWarp = kMaxS / kWarps;   // a multiple of the 16 keys of a k-step

__device__ __forceinline__ uint32_t sm_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ---- bulk-tensor loads (the TMA form) ----
constexpr long long kWaitCycles = 3000000000LL;   // ~1.5 s: a wait that long has failed
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
// tensor-map coordinates of a box: contraction index k, row index r, (batch, head) index bz split as (bz / b0, bz % b0)
__device__ __forceinline__ void box_coords(const int* sel, int k, int r, int bz, int b0, int* c) {
  const int lo = bz % b0, hi = bz / b0;
#pragma unroll
  for (int d = 0; d < 5; ++d) {
    const int q = sel[d];
    c[d] = q == 0 ? k : q == 2 ? r : q == 4 ? lo : q == 5 ? hi : 0;
  }
}

// TMA = false: Q, K and V arrive by per-thread cp.async into rows padded by 16 bytes. TMA = true: by bulk-tensor loads of
// 64-row x 128-byte boxes with the 128-byte swizzle (the tensor maps the tensor-memory forms use), one thread issuing
// them all: Q and K complete on one mbarrier, V on a second that is waited for only before P.V. A tile is then
// [64-column chunk of d][64-key half][64 rows][128 bytes], 16-byte piece c of row r at piece c ^ (r % 8).
template <int D, bool TMA>
__device__ __forceinline__ void attn_small_body(const AttnParams& p, const CUtensorMap* mq, const CUtensorMap* mk, const CUtensorMap* mv) {
  constexpr int PITCH = D * 2 + 16;   // bytes per shared-memory row (cp.async form): 16 bytes of padding keep ldmatrix's eight rows on distinct banks
  constexpr int CPR = D / 8;          // 16-byte pieces per row
  constexpr int DW = D / kWarps;      // output columns per warp
  constexpr int DC = D / 64;          // 64-column chunks of the head dim (TMA form: one box column each)
  extern __shared__ __align__(1024) uint8_t smem[];
  pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_qt = (p.S + kRowsPerCta - 1) / kRowsPerCta;
  const int qt = int(blockIdx.x) % n_qt, bz = int(blockIdx.x) / n_qt;
  const int h = bz % p.NH, b = bz / p.NH;
  const int m0 = qt * kRowsPerCta;
  // keys this CTA needs (a causal mask hides those past its last query), rounded up to the 16 of a k-step
  const int s_cta = p.causal ? min(p.S, m0 + kRowsPerCta) : p.S;
  const int s_pad = (s_cta + 15) & ~15;
  const int n_k16 = s_pad >> 4;
  // the cp.async form: Q | P | maxima, sums | K | V (rows of PITCH bytes); the TMA form: Q | K | V (boxes) | P | maxima, sums | barriers
  uint8_t* sQ = smem;
  uint8_t* sK = TMA ? sQ + DC * 8192 : sQ + kRowsPerCta * PITCH + kRowsPerCta * kPPitch + 2 * kWarps * kRowsPerCta * int(sizeof(float));
  uint8_t* sV = TMA ? sK + DC * 16384 : sK + s_pad * PITCH;
  uint8_t* sP = TMA ? sV + DC * 16384 : sQ + kRowsPerCta * PITCH;
  float* xm = reinterpret_cast<float*>(sP + kRowsPerCta * kPPitch);   // [warp][row] maxima
  float* xl = xm + kWarps * kRowsPerCta;                               // [warp][row] sums
  const uint32_t bars = sm_addr(xl + kWarps * kRowsPerCta);            // TMA form: two mbarriers
  // shared-memory address of 16-byte piece c of row r of Q, and of key `key` of K / V
  auto q_at = [&](int r, int c) -> uint32_t {
    return TMA ? sm_addr(sQ) + uint32_t((c >> 3) * 8192 + r * 128 + (((c & 7) ^ (r & 7)) << 4))
               : sm_addr(sQ) + uint32_t(r * PITCH + c * 16);
  };
  auto kv_at = [&](const uint8_t* base, int key, int c) -> uint32_t {
    return TMA ? sm_addr(base) + uint32_t((c >> 3) * 16384 + (key >> 6) * 8192 + (key & 63) * 128 + (((c & 7) ^ (key & 7)) << 4))
               : sm_addr(base) + uint32_t(key * PITCH + c * 16);
  };
  bool loads_ok = true;
  if constexpr (TMA) {
    if (sm_addr(smem) & 1023u) {   // cannot happen with the launch this file does; refuse rather than read misplaced boxes
      if (tid == 0) atomicOr(p.status, 0x100u | 0x08u);
      return;
    }
    if (tid == 0) {
      mbar_init(bars, 1);
      mbar_init(bars + 8, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();   // Q, K, V come from the previous steps; O may still be read by an earlier one
    if (tid == 0) {
      const int halves = s_pad > 64 ? 2 : 1;   // 64-key boxes; keys past the sequence arrive as zeros
      int c[5];
      mbar_expect_tx(bars, uint32_t(DC + DC * halves) * 8192u);
      for (int dc = 0; dc < DC; ++dc) {
        box_coords(p.q_sel, dc * 64, m0, bz, p.q_b0, c);
        tma_load5(sm_addr(sQ) + dc * 8192, mq, bars, c);
        for (int hf = 0; hf < halves; ++hf) {
          box_coords(p.k_sel, dc * 64, hf * 64, bz, p.k_b0, c);
          tma_load5(sm_addr(sK) + dc * 16384 + hf * 8192, mk, bars, c);
        }
      }
      mbar_expect_tx(bars + 8, uint32_t(DC * halves) * 8192u);
      for (int dc = 0; dc < DC; ++dc)
        for (int hf = 0; hf < halves; ++hf) {
          box_coords(p.v_sel, hf * 64, dc * 64, bz, p.v_b0, c);   // V as the second product's operand: rows are d, the contraction runs over keys
          tma_load5(sm_addr(sV) + dc * 16384 + hf * 8192, mv, bars + 8, c);
        }
    }
    loads_ok = mbar_wait(bars, 0);   // Q and K have landed; V is still on its way
  } else {
    const __nv_bfloat16* Qg = static_cast<const __nv_bfloat16*>(p.Q) + (int64_t)b * p.q_s[0] + (int64_t)h * p.q_s[1];
    const __nv_bfloat16* Kg = static_cast<const __nv_bfloat16*>(p.K) + (int64_t)b * p.k_s[0] + (int64_t)h * p.k_s[1];
    const __nv_bfloat16* Vg = static_cast<const __nv_bfloat16*>(p.V) + (int64_t)b * p.v_s[0] + (int64_t)h * p.v_s[1];
    pdl_wait();   // Q, K, V come from the previous steps; O may still be read by an earlier one
    // rows past the sequence are zero-filled: a zero probability times whatever lay there would not be zero
    for (int i = tid; i < kRowsPerCta * CPR; i += 32 * kWarps) {
      const int row = i / CPR, c = i - row * CPR;
      uint8_t* dst = sQ + row * PITCH + c * 16;
      if (m0 + row < p.S) cp_async16(sm_addr(dst), Qg + (int64_t)(m0 + row) * p.q_s[2] + c * 8);
      else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
    }
    for (int i = tid; i < s_pad * CPR; i += 32 * kWarps) {
      const int row = i / CPR, c = i - row * CPR;
      uint8_t* dk = sK + row * PITCH + c * 16;
      if (row < p.S) cp_async16(sm_addr(dk), Kg + (int64_t)row * p.k_s[2] + c * 8);
      else *reinterpret_cast<uint4*>(dk) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int i = tid; i < s_pad * CPR; i += 32 * kWarps) {
      const int row = i / CPR, c = i - row * CPR;
      uint8_t* dv = sV + row * PITCH + c * 16;
      if (row < p.S) cp_async16(sm_addr(dv), Vg + (int64_t)row * p.v_s[2] + c * 8);
      else *reinterpret_cast<uint4*>(dv) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // Q and K have landed; V is still on its way
    __syncthreads();
  }

  const int quad = lane >> 2, qlane = lane & 3;
  // ---- S = Q.K^T for this warp's keys: 16 rows x kKeysPerWarp keys, fp32, in registers ----
  constexpr int NT = kKeysPerWarp / 8;  // 8-key n-tiles per warp
  float sc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
  const int key0 = warp * kKeysPerWarp;
  if (key0 < s_pad && loads_ok) {       // (uniform across the warp) otherwise every score of this warp is masked
    const int q_row = (lane & 7) + ((lane >> 3) & 1) * 8;
    // lane l addresses matrix l / 8: keys 8 (l / 16) + l % 8 of a 16-key pair of n-tiles, d half (l / 8) % 2
    const int k_key = key0 + (lane >> 4) * 8 + (lane & 7);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      uint32_t a0, a1, a2, a3;
      ldsm_x4(q_at(q_row, kk * 2 + (lane >> 4)), a0, a1, a2, a3);
#pragma unroll
      for (int j = 0; j < NT / 2; ++j) {
        if (key0 + 16 * j < s_pad) {    // (uniform) pairs past the keys this CTA needs stay zero and are masked below
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kv_at(sK, k_key + 16 * j, kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
          mma_bf16(sc[2 * j], a0, a1, a2, a3, b0, b1);
          mma_bf16(sc[2 * j + 1], a0, a1, a2, a3, b2, b3);
        }
      }
    }
  }
  // ---- softmax: this thread holds rows quad and quad + 8, keys key0 + 8 nt + 2 qlane + {0, 1} ----
  const int q0 = m0 + quad, q1 = q0 + 8;
  const int lim0 = p.causal ? min(p.S, q0 + 1) : p.S, lim1 = p.causal ? min(p.S, q1 + 1) : p.S;   // keys >= lim are masked
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int kc = key0 + nt * 8 + qlane * 2;
    if (kc >= lim0) sc[nt][0] = -INFINITY;
    if (kc + 1 >= lim0) sc[nt][1] = -INFINITY;
    if (kc >= lim1) sc[nt][2] = -INFINITY;
    if (kc + 1 >= lim1) sc[nt][3] = -INFINITY;
    mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
    mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
  }
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  if (qlane == 0) { xm[warp * kRowsPerCta + quad] = mx0; xm[warp * kRowsPerCta + quad + 8] = mx1; }
  __syncthreads();
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    mx0 = fmaxf(mx0, xm[w * kRowsPerCta + quad]);
    mx1 = fmaxf(mx1, xm[w * kRowsPerCta + quad + 8]);
  }
  // a row past the sequence has no visible key: any finite reference point keeps it free of NaNs (it is not stored)
  const float nm0 = mx0 == -INFINITY ? 0.f : -ceilf(mx0 * p.scale_log2);
  const float nm1 = mx1 == -INFINITY ? 0.f : -ceilf(mx1 * p.scale_log2);
  float l0 = 0.f, l1 = 0.f;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const float e0 = ex2_approx(fmaf(sc[nt][0], p.scale_log2, nm0)), e1 = ex2_approx(fmaf(sc[nt][1], p.scale_log2, nm0));
    const float e2 = ex2_approx(fmaf(sc[nt][2], p.scale_log2, nm1)), e3 = ex2_approx(fmaf(sc[nt][3], p.scale_log2, nm1));
    l0 += e0 + e1;
    l1 += e2 + e3;
    // P[row][key] as bf16, row-major, for the A fragments of the second product
    const int kc = key0 + nt * 8 + qlane * 2;
    *reinterpret_cast<uint32_t*>(sP + quad * kPPitch + kc * 2) = pack_bf16(e0, e1);
    *reinterpret_cast<uint32_t*>(sP + (quad + 8) * kPPitch + kc * 2) = pack_bf16(e2, e3);
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  if (qlane == 0) { xl[warp * kRowsPerCta + quad] = l0; xl[warp * kRowsPerCta + quad + 8] = l1; }
  if constexpr (TMA) {
    if (loads_ok) loads_ok = mbar_wait(bars + 8, 0);       // V has landed
    else mbar_wait(bars + 8, 0);                          // (give the copies in flight their time before the memory is given up)
  } else {
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // this thread's pieces of V
  }
  __syncthreads();                                        // everybody's P, sums and pieces of V
  if (!loads_ok) {                                        // a bounded wait gave up: report, store nothing
    if (lane == 0) atomicOr(p.status, 0x100u | 0x1000u);
    return;
  }

  // ---- O = P.V for this warp's output columns DW w .. DW w + DW - 1 ----
  float oc[DW / 8][4];
#pragma unroll
  for (int nt = 0; nt < DW / 8; ++nt) oc[nt][0] = oc[nt][1] = oc[nt][2] = oc[nt][3] = 0.f;
  {
    const uint32_t p_lane = sm_addr(sP) + uint32_t(((lane & 7) + ((lane >> 3) & 1) * 8) * kPPitch + (lane >> 4) * 16);
    // transposed 8 x 8 loads: lane l addresses matrix l / 8: keys 8 ((l / 8) % 2) + l % 8 of the k-step, d tile l / 16 of a pair
    const int v_key = ((lane >> 3) & 1) * 8 + (lane & 7);
    const int v_c = warp * DW / 8 + (lane >> 4);
#pragma unroll
    for (int j = 0; j < kMaxS / 16; ++j) {
      if (j < n_k16) {
        uint32_t a0, a1, a2, a3;
        ldsm_x4(p_lane + j * 32, a0, a1, a2, a3);
#pragma unroll
        for (int np = 0; np < DW / 16; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(kv_at(sV, v_key + 16 * j, v_c + 2 * np), b0, b1, b2, b3);
          mma_bf16(oc[2 * np], a0, a1, a2, a3, b0, b1);
          mma_bf16(oc[2 * np + 1], a0, a1, a2, a3, b2, b3);
        }
      }
    }
  }
  // ---- O / l -> bf16 ----
  l0 = 0.f; l1 = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    l0 += xl[w * kRowsPerCta + quad];
    l1 += xl[w * kRowsPerCta + quad + 8];
  }
  const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
  __nv_bfloat16* og = static_cast<__nv_bfloat16*>(p.O) + (int64_t)b * p.o_s[0] + (int64_t)h * p.o_s[1];
#pragma unroll
  for (int nt = 0; nt < DW / 8; ++nt) {
    const int d = warp * DW + nt * 8 + qlane * 2;
    if (q0 < p.S) *reinterpret_cast<uint32_t*>(og + (int64_t)q0 * p.o_s[2] + d) = pack_bf16(oc[nt][0] * i0, oc[nt][1] * i0);
    if (q1 < p.S) *reinterpret_cast<uint32_t*>(og + (int64_t)q1 * p.o_s[2] + d) = pack_bf16(oc[nt][2] * i1, oc[nt][3] * i1);
  }
}


template <int D>
__global__ void __launch_bounds__(32 * kWarps) attn_small_kernel(const AttnParams p) {
  attn_small_body<D, false>(p, nullptr, nullptr, nullptr);
}
template <int D>
__global__ void __launch_bounds__(32 * kWarps) attn_small_tma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                                                                     const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  attn_small_body<D, true>(p, &map_q, &map_k, &map_v);
}

}  // namespace

bool attn_small_eligible(const AttnParams& p) {
  return p.rows_d_contiguous && p.S >= 1 && p.S <= kMaxS && (p.D == 64 || p.D == 128) && p.Q && p.K && p.V && p.O &&
         !((reinterpret_cast<uintptr_t>(p.Q) | reinterpret_cast<uintptr_t>(p.K) | reinterpret_cast<uintptr_t>(p.V)) & 15) &&
         !(reinterpret_cast<uintptr_t>(p.O) & 3);
}

static size_t attn_small_smem(int D, int s_pad) {
  return size_t(kRowsPerCta + 2 * s_pad) * (D * 2 + 16) + size_t(kRowsPerCta) * kPPitch + size_t(2) * kWarps * kRowsPerCta * sizeof(float);
}
static size_t attn_small_tma_smem(int D) {
  return size_t(D / 64) * (8192 + 2 * 16384) + size_t(kRowsPerCta) * kPPitch + size_t(2) * kWarps * kRowsPerCta * sizeof(float) + 16;
}
// FLUID_ATTN_SMALL_TMA=0 in the environment keeps the loads on per-thread cp.async (A/B timing).
static bool small_tma_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("FLUID_ATTN_SMALL_TMA");
    return !(e && e[0] == '0');
  }();
  return on;
}

cudaError_t launch_attn_small(const AttnParams& p, const AttnHost* host, cudaStream_t stream) {
  const int s_pad = (p.S + 15) & ~15;   // (a causal CTA may need fewer rows; the launch reserves the most any CTA uses)
  const dim3 grid(((p.S + kRowsPerCta - 1) / kRowsPerCta) * p.B * p.NH);
  static bool attr[4] = {false, false, false, false};
  auto set_attr = [&](int slot, const void* fn, size_t bytes) -> cudaError_t {
    if (attr[slot]) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
    if (e == cudaSuccess) attr[slot] = true;
    return e;
  };
  if (host && host->eligible && small_tma_enabled()) {
    const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(&host->map_q);
    const CUtensorMap* mk = reinterpret_cast<const CUtensorMap*>(&host->map_k);
    const CUtensorMap* mv = reinterpret_cast<const CUtensorMap*>(&host->map_v);
    const size_t smem = attn_small_tma_smem(p.D);
    if (p.D == 64) {
      cudaError_t e = set_attr(2, reinterpret_cast<const void*>(attn_small_tma_kernel<64>), smem);
      if (e != cudaSuccess) return e;
      return launch_k(attn_small_tma_kernel<64>, grid, 32 * kWarps, smem, stream, *mq, *mk, *mv, p);
    }
    cudaError_t e = set_attr(3, reinterpret_cast<const void*>(attn_small_tma_kernel<128>), smem);
    if (e != cudaSuccess) return e;
    return launch_k(attn_small_tma_kernel<128>, grid, 32 * kWarps, smem, stream, *mq, *mk, *mv, p);
  }
  const size_t smem = attn_small_smem(p.D, s_pad);
  if (p.D == 64) {
    cudaError_t e = set_attr(0, reinterpret_cast<const void*>(attn_small_kernel<64>), attn_small_smem(64, kMaxS));
    if (e != cudaSuccess) return e;
    return launch_k(attn_small_kernel<64>, grid, 32 * kWarps, smem, stream, p);
  }
  cudaError_t e = set_attr(1, reinterpret_cast<const void*>(attn_small_kernel<128>), attn_small_smem(128, kMaxS));
  if (e != cudaSuccess) return e;
  return launch_k(attn_small_kernel<128>, grid, 32 * kWarps, smem, stream, p);
}

}  // namespace fluid
