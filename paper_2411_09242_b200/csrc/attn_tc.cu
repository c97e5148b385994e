// Fused attention for sm_100a: S = Q.K^T and O = softmax(S).V on tcgen05 tensor cores with the
// score tile kept in tensor memory; the [S, S] score / probability tensors never reach HBM or the
// arena. One CTA = one (batch, head, 128-query tile); 256 threads: two per query row, each owning
// half of the key columns of a tile (two warps per scheduler hide each other's latencies).
//
//   per 128-key tile:  TMA K, V tiles (2-stage ring)  ->  tcgen05.mma  S = Q.K^T  (TMEM, fp32)
//                      -> tcgen05.ld, online softmax in registers (row max / sum per thread, exp2)
//                      -> P (bf16) written to shared memory in the 128-byte-swizzled K-major form
//                      -> tcgen05.mma  PV = P.V (TMEM)  ->  O = O * alpha + PV in registers
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

template <int D>
__global__ void __launch_bounds__(256, D == 64 ? 2 : 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const __grid_constant__ AttnParams p) {
  constexpr int DC = D / 64;                       // 64-wide chunks of the head dim
  constexpr uint32_t kTile = TQ * D * 2;           // bytes of one Q / K / V tile
  constexpr uint32_t kPBytes = TQ * TK * 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = sQ + kTile, sV = sK + 2 * kTile, sP = sV + 2 * kTile, bars = sP + kPBytes;
  const uint32_t bar_q = bars, bar_kv0 = bars + 8, bar_s = bars + 24, bar_o = bars + 32, tmem_slot = bars + 40;
  float* xch = reinterpret_cast<float*>(smem_raw + (bars + 64 - raw));   // [2][128] row-max / row-sum exchange
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  uint8_t* p_smem = smem_raw + (sP - raw);

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, row = threadIdx.x & 127, half = threadIdx.x >> 7;
  // CTAs are issued heaviest first: with a causal mask the last query tiles see the most key tiles,
  // so they start first and the short ones fill the gaps (longest-processing-time order)
  const int n_bz = p.B * p.NH;
  const int mt = (int(gridDim.x) / n_bz - 1) - int(blockIdx.x) / n_bz, bz = int(blockIdx.x) % n_bz;
  const int h = bz % p.NH, b = bz / p.NH;
  const int m0 = mt * TQ, qi = m0 + row;
  int n_kv = (p.S + TK - 1) / TK;
  if (p.causal) n_kv = min(n_kv, (m0 + TQ - 1) / TK + 1);

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_kv0, 1); mbar_init(bar_kv0 + 8, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  const uint32_t tS = tmem_base, tO = tmem_base + TK;     // score columns, then PV columns
  const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;   // warps w and w+4 share a lane quarter

  pdl_wait();  // Q, K, V come from the previous steps

  // ---- loads (thread 0) ----
  bool pending[2] = {false, false};   // thread 0: loads issued into a stage and not yet waited for
  auto load_kv = [&](int j, int st) {
    pending[st] = true;
    const uint32_t bar = bar_kv0 + 8u * st;
    mbar_expect_tx(bar, 2 * kTile);
    const int kv0 = j * TK;
    int c[5];
    const uint32_t k_dst = sK + st * kTile, v_dst = sV + st * kTile;
    if (!p.k_mn_major) {          // [d chunk][128 keys][64 d]
      for (int dc = 0; dc < DC; ++dc)
        for (int rh = 0; rh < 2; ++rh) {
          coords(p.k_sel, dc * 64, kv0 + rh * 64, bz, p.k_b0, c);
          tma_load5(k_dst + dc * 16384u + rh * 8192u, &map_k, bar, c);
        }
    } else {                      // [key chunk][D d-rows][64 keys]
      for (int sc = 0; sc < 2; ++sc)
        for (int dc = 0; dc < DC; ++dc) {
          coords(p.k_sel, dc * 64, kv0 + sc * 64, bz, p.k_b0, c);
          tma_load5(k_dst + sc * (D * 128u) + dc * 8192u, &map_k, bar, c);
        }
    }
    if (!p.v_k_major) {           // [d chunk][128 keys][64 d]  (MN-major B of P.V)
      for (int dc = 0; dc < DC; ++dc)
        for (int kc = 0; kc < 2; ++kc) {
          coords(p.v_sel, kv0 + kc * 64, dc * 64, bz, p.v_b0, c);
          tma_load5(v_dst + dc * 16384u + kc * 8192u, &map_v, bar, c);
        }
    } else {                      // [key chunk][D d-rows][64 keys]  (K-major B of P.V)
      for (int kc = 0; kc < 2; ++kc)
        for (int dh = 0; dh < DC; ++dh) {
          coords(p.v_sel, kv0 + kc * 64, dh * 64, bz, p.v_b0, c);
          tma_load5(v_dst + kc * (D * 128u) + dh * 8192u, &map_v, bar, c);
        }
    }
  };
  if (threadIdx.x == 0) {
    mbar_expect_tx(bar_q, kTile);
    int c[5];
    for (int dc = 0; dc < DC; ++dc)
      for (int rh = 0; rh < 2; ++rh) {
        coords(p.q_sel, dc * 64, m0 + rh * 64, bz, p.q_b0, c);
        tma_load5(sQ + dc * 16384u + rh * 8192u, &map_q, bar_q, c);
      }
    load_kv(0, 0);
    if (n_kv > 1) load_kv(1, 1);
  }

  const uint32_t idesc_s = make_idesc(TK, 0, p.k_mn_major);
  const uint32_t idesc_o = make_idesc(D, 0, p.v_k_major ? 0 : 1);
  // m_used is the (possibly stale) row maximum the exponentials are taken against; O (in tensor
  // memory) and l are rescaled only when the true maximum has moved by more than 2^8, so most
  // key tiles accumulate P.V straight into tensor memory with no traffic on O at all.
  float m_used = -INFINITY, l_run = 0.f;
  bool ok = true;
  uint32_t fail = 0;

  auto issue_qk = [&](int j) {   // thread 0: S = Q.K_j^T
    const int st = j & 1;
    if (!mbar_wait(bar_kv0 + 8u * st, uint32_t(j >> 1) & 1u)) { fail |= 0x20u; return; }
    pending[st] = false;
    tc_fence_after();
    const uint32_t kb = sK + st * kTile;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const uint64_t ad = make_desc(sQ + (kk >> 2) * 16384u + (kk & 3) * 32u, 16, 1024);
      const uint64_t bd = p.k_mn_major ? make_desc(kb + kk * 2048u, D * 128u, 1024)
                                       : make_desc(kb + (kk >> 2) * 16384u + (kk & 3) * 32u, 16, 1024);
      umma_bf16(tS, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
    }
    umma_commit(bar_s);
  };

  if (!mbar_wait(bar_q, 0)) { ok = false; fail = 0x10u; }
  ok = __syncthreads_and(ok);
  if (ok && threadIdx.x == 0) issue_qk(0);
  for (int j = 0; ok && j < n_kv; ++j) {
    const int st = j & 1;
    const uint32_t ph = uint32_t(j) & 1u;
    const int kv0 = j * TK;
    if (!mbar_wait(bar_s, ph)) { ok = false; fail |= 0x40u; }
    ok = __syncthreads_and(ok);   // leave the loop together
    if (!ok) break;
    tc_fence_after();
    // ---- this thread owns half (64 columns) of query row qi: read its scores once ----
    constexpr int HC = TK / 2;
    const int cbase = half * HC;
    uint32_t r[HC];
#pragma unroll
    for (int c0 = 0; c0 < HC; c0 += 32) tmem_ld32(tS + lane_addr + cbase + c0, *reinterpret_cast<uint32_t(*)[32]>(&r[c0]));
    tmem_ld_wait();
    const int kv_lim = (p.causal ? min(p.S, qi + 1) : p.S) - kv0 - cbase;   // local columns >= kv_lim are masked
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < HC; ++i)
      if (i < kv_lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
    xch[half * 128 + row] = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
    // the previous tile's P.V must be done before O is rescaled or P / the K,V stage are reused
    if (j > 0) {
      if (!mbar_wait(bar_o, uint32_t(j - 1) & 1u)) { ok = false; fail |= 0x80u; }
      tc_fence_after();
    }
    __syncthreads();
    const float m_tile = fmaxf(xch[row], xch[128 + row]) * p.scale_log2;
    if (j == 0) {
      m_used = m_tile;
    } else {
      const bool need = m_tile > m_used + 8.f;
      if (__any_sync(0xffffffffu, need)) {
        const float m_new = need ? m_tile : m_used;
        const float alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - m_new);
#pragma unroll 1
        for (int c0 = half * (D / 2); c0 < (half + 1) * (D / 2); c0 += 32) {
          uint32_t q[32];
          tmem_ld32(tO + lane_addr + c0, q);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) q[i] = __float_as_uint(__uint_as_float(q[i]) * alpha);
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
              "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
              "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
              ::"r"(tO + lane_addr + c0), "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]), "r"(q[4]), "r"(q[5]), "r"(q[6]),
              "r"(q[7]), "r"(q[8]), "r"(q[9]), "r"(q[10]), "r"(q[11]), "r"(q[12]), "r"(q[13]), "r"(q[14]), "r"(q[15]),
              "r"(q[16]), "r"(q[17]), "r"(q[18]), "r"(q[19]), "r"(q[20]), "r"(q[21]), "r"(q[22]), "r"(q[23]), "r"(q[24]),
              "r"(q[25]), "r"(q[26]), "r"(q[27]), "r"(q[28]), "r"(q[29]), "r"(q[30]), "r"(q[31])
              : "memory");
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        l_run *= alpha;
        m_used = m_new;
      }
    }
    // K/V stage of tile j-1 is free: fetch tile j+1 into it
    if (threadIdx.x == 0 && j >= 1 && j + 1 < n_kv) load_kv(j + 1, (j + 1) & 1);
    // ---- P = exp2(s * k - m_used), bf16, into the swizzled K-major tile (this thread's 64 columns
    //      are exactly one 64-column chunk of the tile) ----
    float ps4[4] = {0.f, 0.f, 0.f, 0.f};
    const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
#pragma unroll
    for (int g = 0; g < HC / 8; ++g) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int col = g * 8 + 2 * i;
        float a = 0.f, bb = 0.f;
        if (col < kv_lim) a = exp2f(fmaf(__uint_as_float(r[col]), p.scale_log2, neg_m));
        if (col + 1 < kv_lim) bb = exp2f(fmaf(__uint_as_float(r[col + 1]), p.scale_log2, neg_m));
        const __nv_bfloat162 hv = __floats2bfloat162_rn(a, bb);   // the sum uses what the tensor core multiplies
        ps4[i] += __low2float(hv) + __high2float(hv);
        w[i] = *reinterpret_cast<const uint32_t*>(&hv);
      }
      const uint32_t off = half * 16384u + row * 128u + ((g ^ (row & 7)) << 4);
      *reinterpret_cast<uint4*>(p_smem + off) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    l_run += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);   // partial sum over this thread's columns
    // generic-proxy writes of P -> visible to the tensor core; S has been consumed by every row
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    ok = __syncthreads_and(ok);
    if (!ok) break;
    if (threadIdx.x == 0) {
      tc_fence_after();
      const uint32_t vb = sV + st * kTile;
#pragma unroll
      for (int kk = 0; kk < TK / 16; ++kk) {
        const uint64_t ad = make_desc(sP + (kk >> 2) * 16384u + (kk & 3) * 32u, 16, 1024);
        const uint64_t bd = p.v_k_major ? make_desc(vb + (kk >> 2) * (D * 128u) + (kk & 3) * 32u, 16, 1024)
                                        : make_desc(vb + kk * 2048u, 16384, 1024);
        umma_bf16(tO, ad, bd, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);   // O accumulates across key tiles
      }
      umma_commit(bar_o);
      if (j + 1 < n_kv) issue_qk(j + 1);   // queued behind P.V: ready when the next softmax starts
    }
  }
  // ---- O / l -> bf16 ----
  if (ok && n_kv > 0) {
    if (!mbar_wait(bar_o, uint32_t(n_kv - 1) & 1u)) { ok = false; fail |= 0x80u; }
    tc_fence_after();
  }
  ok = __syncthreads_and(ok);
  if (fail) atomicOr(p.status, 0x100u | fail);
  if (threadIdx.x == 0 && !ok) {   // let loads still in flight land before the shared memory is given up
    for (int st = 0; st < 2; ++st)
      if (pending[st]) mbar_wait(bar_kv0 + 8u * st, 0) || mbar_wait(bar_kv0 + 8u * st, 1);
  }
  xch[half * 128 + row] = l_run;
  __syncthreads();
  if (ok) {
    const float l_tot = xch[row] + xch[128 + row];
    const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.O) + (int64_t)b * p.o_s[0] + (int64_t)h * p.o_s[1] + (int64_t)qi * p.o_s[2];
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
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

}  // namespace

cudaError_t launch_attn_tc(const AttnParams& p, const AttnHost& host, cudaStream_t stream) {
  const int D = p.D;
  const size_t smem = size_t(5) * TQ * D * 2 + size_t(TQ) * TK * 2 + 1024 + 64 + 1024;
  const dim3 grid(((p.S + TQ - 1) / TQ) * p.B * p.NH);
  const CUtensorMap* mq = reinterpret_cast<const CUtensorMap*>(&host.map_q);
  const CUtensorMap* mk = reinterpret_cast<const CUtensorMap*>(&host.map_k);
  const CUtensorMap* mv = reinterpret_cast<const CUtensorMap*>(&host.map_v);
  static bool attr64 = false, attr128 = false;
  if (D == 64) {
    if (!attr64) {
      cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      attr64 = true;
    }
    return launch_k(attn_tc_kernel<64>, grid, 256, smem, stream, *mq, *mk, *mv, p);
  }
  if (D == 128) {
    if (!attr128) {
      cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      attr128 = true;
    }
    return launch_k(attn_tc_kernel<128>, grid, 256, smem, stream, *mq, *mk, *mv, p);
  }
  return cudaErrorInvalidValue;
}

}  // namespace fluid
