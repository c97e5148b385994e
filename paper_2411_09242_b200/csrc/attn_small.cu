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
// slower: 0.483 against 0.477 ms for a twelve-layer encoder step). K arrives first and V in a second
// cp.async group that lands under Q.K^T and the softmax. The tensor cores are only the arithmetic unit.
// Same numeric reading as the other forms: the reference point of the exponentials is the row maximum rounded up to a
// whole number in the base-2 domain, P is rounded to bf16 for the second product, the row sum uses the unrounded
// exponentials, masked entries are exactly zero.
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
__device__ __forceinline__ void ldsm_x2_t(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
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

template <int D>
__global__ void __launch_bounds__(32 * kWarps) attn_small_kernel(const AttnParams p) {
  constexpr int PITCH = D * 2 + 16;   // bytes per shared-memory row: 16 bytes of padding keep ldmatrix's eight rows on distinct banks
  constexpr int CPR = D / 8;          // 16-byte pieces per row
  constexpr int DW = D / kWarps;      // output columns per warp
  extern __shared__ __align__(16) uint8_t smem[];
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
  uint8_t* sQ = smem;
  uint8_t* sP = sQ + kRowsPerCta * PITCH;
  float* xm = reinterpret_cast<float*>(sP + kRowsPerCta * kPPitch);   // [warp][row] maxima
  float* xl = xm + kWarps * kRowsPerCta;                               // [warp][row] sums
  uint8_t* sK = reinterpret_cast<uint8_t*>(xl + kWarps * kRowsPerCta);
  uint8_t* sV = sK + s_pad * PITCH;
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

  const int quad = lane >> 2, qlane = lane & 3;
  // ---- S = Q.K^T for this warp's keys: 16 rows x kKeysPerWarp keys, fp32, in registers ----
  constexpr int NT = kKeysPerWarp / 8;  // 8-key n-tiles per warp
  float sc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
  const int key0 = warp * kKeysPerWarp;
  if (key0 < s_pad) {                   // (uniform across the warp) otherwise every score of this warp is masked
    const uint32_t q_lane = sm_addr(sQ) + uint32_t(((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + (lane >> 4) * 16);
    // lane l addresses matrix l / 8: keys 8 (l / 16) + l % 8 of a 16-key pair of n-tiles, d half (l / 8) % 2
    const uint32_t k_lane = sm_addr(sK) + uint32_t((key0 + (lane >> 4) * 8 + (lane & 7)) * PITCH + ((lane >> 3) & 1) * 16);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      uint32_t a0, a1, a2, a3;
      ldsm_x4(q_lane + kk * 32, a0, a1, a2, a3);
#pragma unroll
      for (int j = 0; j < NT / 2; ++j) {
        if (key0 + 16 * j < s_pad) {    // (uniform) pairs past the keys this CTA needs stay zero and are masked below
          uint32_t b0, b1, b2, b3;
          ldsm_x4(k_lane + uint32_t(j * 16 * PITCH) + kk * 32, b0, b1, b2, b3);
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
  asm volatile("cp.async.wait_group 0;" ::: "memory");   // this thread's pieces of V
  __syncthreads();                                        // everybody's P, sums and pieces of V

  // ---- O = P.V for this warp's output columns DW w .. DW w + DW - 1 ----
  float oc[DW / 8][4];
#pragma unroll
  for (int nt = 0; nt < DW / 8; ++nt) oc[nt][0] = oc[nt][1] = oc[nt][2] = oc[nt][3] = 0.f;
  {
    const uint32_t p_lane = sm_addr(sP) + uint32_t(((lane & 7) + ((lane >> 3) & 1) * 8) * kPPitch + (lane >> 4) * 16);
    // transposed 8 x 8 loads: lane l addresses matrix l / 8: keys 8 ((l / 8) % 2) + l % 8 of the k-step, d tile l / 16 of a
    // pair (with one 8-column tile per warp only lanes 0-15 address a matrix; the others repeat them)
    const uint32_t v_lane = sm_addr(sV) + uint32_t((((lane >> 3) & 1) * 8 + (lane & 7)) * PITCH + (warp * DW * 2) +
                                                   (DW >= 16 ? (lane >> 4) * 16 : 0));
#pragma unroll
    for (int j = 0; j < kMaxS / 16; ++j) {
      if (j < n_k16) {
        uint32_t a0, a1, a2, a3;
        ldsm_x4(p_lane + j * 32, a0, a1, a2, a3);
        if constexpr (DW >= 16) {
#pragma unroll
          for (int np = 0; np < DW / 16; ++np) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(v_lane + uint32_t(j * 16 * PITCH) + np * 32, b0, b1, b2, b3);
            mma_bf16(oc[2 * np], a0, a1, a2, a3, b0, b1);
            mma_bf16(oc[2 * np + 1], a0, a1, a2, a3, b2, b3);
          }
        } else {
          uint32_t b0, b1;
          ldsm_x2_t(v_lane + uint32_t(j * 16 * PITCH), b0, b1);
          mma_bf16(oc[0], a0, a1, a2, a3, b0, b1);
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

}  // namespace

bool attn_small_eligible(const AttnParams& p) {
  return p.rows_d_contiguous && p.S >= 1 && p.S <= kMaxS && (p.D == 64 || p.D == 128) && p.Q && p.K && p.V && p.O &&
         !((reinterpret_cast<uintptr_t>(p.Q) | reinterpret_cast<uintptr_t>(p.K) | reinterpret_cast<uintptr_t>(p.V)) & 15) &&
         !(reinterpret_cast<uintptr_t>(p.O) & 3);
}

static size_t attn_small_smem(int D, int s_pad) {
  return size_t(kRowsPerCta + 2 * s_pad) * (D * 2 + 16) + size_t(kRowsPerCta) * kPPitch + size_t(2) * kWarps * kRowsPerCta * sizeof(float);
}

cudaError_t launch_attn_small(const AttnParams& p, cudaStream_t stream) {
  const int s_pad = (p.S + 15) & ~15;   // (a causal CTA may need fewer rows; the launch reserves the most any CTA uses)
  const size_t smem = attn_small_smem(p.D, s_pad);
  const dim3 grid(((p.S + kRowsPerCta - 1) / kRowsPerCta) * p.B * p.NH);
  static bool attr[2] = {false, false};
  if (p.D == 64) {
    if (!attr[0]) {
      cudaError_t e = cudaFuncSetAttribute(attn_small_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(attn_small_smem(64, kMaxS)));
      if (e != cudaSuccess) return e;
      attr[0] = true;
    }
    return launch_k(attn_small_kernel<64>, grid, 32 * kWarps, smem, stream, p);
  }
  if (!attr[1]) {
    cudaError_t e = cudaFuncSetAttribute(attn_small_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(attn_small_smem(128, kMaxS)));
    if (e != cudaSuccess) return e;
    attr[1] = true;
  }
  return launch_k(attn_small_kernel<128>, grid, 32 * kWarps, smem, stream, p);
}

}  // namespace fluid
