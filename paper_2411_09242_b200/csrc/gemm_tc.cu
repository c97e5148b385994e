// Tensor-core GEMM for sm_100a: TMA-fed shared-memory ring, tcgen05.mma with fp32 accumulators in
// tensor memory, warp-specialised persistent CTAs (one per SM).
//
//   warp 0      TMA producer: one elected thread issues cp.async.bulk.tensor loads of the A and B
//               tiles of each k-step into a ring of shared-memory stages (mbarrier complete_tx)
//   warp 1      allocates tensor memory; one elected thread issues tcgen05.mma (128 x BN x 16 per
//               instruction, four per stage) and commits stage-release / accumulator-ready barriers
//   warps 2-9   epilogue: tcgen05.ld the accumulator (one row per thread), apply
//               scale / bias / GELU / residual in fp32, store in whatever layout the plan chose
//
// Two accumulators (2 x BN tensor-memory columns) let the epilogue of tile i overlap the MMAs of
// tile i+1. Operands may be K-major or MN-major in global memory (row-/column-/head-major
// tensors): the TMA box and the shared-memory matrix descriptor follow the operand's major, so
// no transpose kernel ever runs. No load uses cluster multicast; the only multicast is the cta_group::2
// tcgen05.commit that arrives on both CTAs' mbarriers of a pair.
//
// Every wait is bounded: a wait that does not complete within about a second records a code in
// the arena header and the CTA drains and exits; the host reads the code with fluid_status().
#include <cuda.h>

#include <algorithm>
#include <cstdlib>
#include <cstdio>

#include <mutex>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

void set_error(const char* fmt, ...);

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t kATileBytes = BM * BK * 2;
constexpr long long kWaitCycles = 3000000000LL;  // ~1.5 s at 2 GHz

struct TcParams {
  GemmParams g;      // group 0 (shapes, A strides, flags are common to all groups)
  GemmParams gx[2];  // groups 1, 2: own B, C, bias and C strides
  int n_group;
  int tiles_per_group;
  GemmTcCfg cfg;
  int tiles_m, tiles_n;
  int num_tiles;        // work items = output tiles x split_k
  int tiles_per_batch;
  int split_k;          // >1: each output tile's k range is cut in split_k pieces run by different CTAs
  int ksteps_per_split;
  float* partial;       // split-K scratch: [tile][split][bn/4][128 rows][4] fp32
  uint32_t* status;     // word 0: device status; words 8..63: per-tile arrival counters for split-K
  int scalar_turn;      // general epilogue: n is contiguous and unsplit in C (and R), so the shared-memory turn applies
  int swiglu;           // CTA-pair form: CTA 0 loads gate columns, CTA 1 up columns; the epilogue writes SiLU(gate) * up
  RopeFreq rope_freq;   // CTA-pair form with a rotary epilogue (groups whose GemmParams has rope = 1)
};

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete in time (the caller records it and drains).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255) == 0 && clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
// The same wait with one answer for the whole warp, for code that goes on to warp-synchronous instructions
// (tcgen05.ld, named barriers): each lane times its own wait, so without the vote a barrier that completes right
// at the limit could let some lanes pass and others give up.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity));
}

// Every tensor map is padded to rank 5 (unit dims), so one instruction form serves all operands.
__device__ __forceinline__ void tma_load(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                         int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Each descriptor is given as its two 32-bit halves: only the low word (the 16-byte-unit address
// field) moves from MMA to MMA, so the issuing thread does 32-bit arithmetic only.
__device__ __forceinline__ void umma_bf16_lohi(uint32_t tmem_c, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                               uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n .reg .b64 da, db;\n mov.b64 da, {%1, %2};\n mov.b64 db, {%3, %4};\n setp.ne.b32 p, %6, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n}"
      ::"r"(tmem_c), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
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
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void sts128(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// The same without the compiler-level memory clobber, for reads that follow a barrier wait (itself a
// volatile statement with a clobber) and must not force every cached parameter to be re-read.
__device__ __forceinline__ float4 lds128_relaxed(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}

// Shared-memory matrix descriptor, 128-byte swizzle. K-major: rows of 128 bytes, 8-row groups
// 1024 bytes apart. MN-major: 64-element chunks of the row index 8192 bytes apart (one chunk =
// 64 k-rows of 128 bytes), 8-k groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, bool mn_major) {
  const uint64_t lbo = mn_major ? (8192 >> 4) : 1;
  const uint64_t sbo = 1024 >> 4;
  return uint64_t((saddr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);
}

__device__ __forceinline__ uint32_t make_idesc(int bn, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn) << 15) | (uint32_t(b_mn) << 16) |
         (uint32_t(bn >> 3) << 17) | (uint32_t(BM >> 4) << 24);
}

// i -> (i / x0, i % x0) without a division in the common merged case (x0 > i)
__device__ __forceinline__ void split2(int i, int x0, int& hi, int& lo) {
  if (i < x0) { hi = 0; lo = i; }
  else { hi = i / x0; lo = i - hi * x0; }
}

// Tile index -> (batch, m tile, n tile); m runs fastest so that CTAs running together share the
// B tile. With CAUSAL_SKIP_UPPER only tiles that touch the lower triangle are enumerated.
__device__ __forceinline__ void decode_tile(const TcParams& p, int tile, int& grp, int& bz, int& mt, int& nt) {
  int r;
  split2(tile, p.tiles_per_group, grp, r);
  split2(r, p.tiles_per_batch, bz, r);
  if (p.g.causal == CAUSAL_SKIP_UPPER) {
    for (int m = 0; m < p.tiles_m; ++m) {
      const int nv = min(p.tiles_n, (m * BM + BM - 1) / p.cfg.bn + 1);
      if (r < nv) { mt = m; nt = r; return; }
      r -= nv;
    }
    mt = 0; nt = 0;
    return;
  }
  split2(r, p.tiles_m, nt, mt);
}

__device__ __forceinline__ int k_steps_of(const TcParams& p, int mt) {
  int kend = p.g.K;
  if (p.g.causal == CAUSAL_CLIP_K) kend = min(kend, mt * BM + BM);
  return (kend + BK - 1) / BK;
}

// work item -> output tile and its k-step range [k_begin, k_begin + count)
template <bool SPLIT>
__device__ __forceinline__ void decode_item(const TcParams& p, int item, int& tile, int& sp, int& k_begin, int& count) {
  if (!SPLIT) { tile = item; sp = 0; k_begin = 0; count = -1; return; }
  tile = item / p.split_k;
  sp = item - tile * p.split_k;
  const int total = (p.g.K + BK - 1) / BK;
  k_begin = sp * p.ksteps_per_split;
  count = min(p.ksteps_per_split, total - k_begin);
}

__device__ __forceinline__ void fill_coords(const int* sel, int rank, int k0, int k1, int r0, int r1, int b0, int b1, int* c) {
#pragma unroll
  for (int d = 0; d < 5; ++d) {
    const int q = sel[d];
    c[d] = q == 0 ? k0 : q == 1 ? k1 : q == 2 ? r0 : q == 3 ? r1 : q == 4 ? b0 : q == 5 ? b1 : 0;
  }
}

__device__ __forceinline__ int64_t split_off(int i, int x0, int64_t s1, int64_t s0) {
  int hi, lo;
  split2(i, x0, hi, lo);
  return (int64_t)hi * s1 + (int64_t)lo * s0;
}


template <int ACT>
__device__ __forceinline__ float act_t(float v) {
  if (ACT == ACT_GELU_ERF) return gelu_erf_fast(v);
  if (ACT == ACT_GELU_TANH) return gelu_tanh(v);
  return v;
}
// the activation of two values (the erf GELU as packed instructions)
template <int ACT>
__device__ __forceinline__ void act2_t(float& a, float& b) {
  if (ACT == ACT_GELU_ERF) { gelu_erf_fast2(a, b); return; }
  a = act_t<ACT>(a);
  b = act_t<ACT>(b);
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}

// Vector epilogue for one 32-column chunk of one accumulator row. Preconditions (checked on the
// host): the n index is contiguous in C (and R), every 8-column group is 16-byte aligned and
// never straddles an n split, N is a multiple of 8.
// With `partial` set (the last-arriving CTA of a split-K tile) the accumulator chunk is the sum, in
// split order, of the partial tiles in scratch memory instead of a tensor-memory load.
template <int ACT, bool HAS_RES, bool C_WIDE, bool R_WIDE>
__device__ __forceinline__ void epilogue_chunk_vec(const GemmParams& g, uint32_t taddr, bool row_ok, int64_t cb,
                                                   int64_t rb, int n, const float* partial = nullptr, int split_k = 1,
                                                   size_t split_stride = 0) {
  uint32_t r[32];
  if (!partial) tmem_ld32(taddr, r);
  // group offsets (an 8-column group shares one n split)
  int64_t co[4], ro[4];
  int n1, n0i;
  split2(n, g.N0, n1, n0i);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    co[q] = cb + (int64_t)n1 * g.c_s[4] + n0i;
    ro[q] = HAS_RES ? rb + (int64_t)n1 * g.r_s[4] + n0i : 0;
    n0i += 8;
    if (n0i >= g.N0) { n0i -= g.N0; ++n1; }
  }
  // operands that do not depend on the accumulator are fetched while the tensor-memory load flies
  uint4 bq[4];
  uint4 rq[HAS_RES ? (R_WIDE ? 8 : 4) : 1];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const bool live = n + 8 * q < g.N;
    if (g.has_bias) bq[q] = live ? *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(g.bias) + n + 8 * q) : make_uint4(0, 0, 0, 0);
    if (HAS_RES && row_ok && live) {
      if (R_WIDE) {
        rq[2 * q] = *reinterpret_cast<const uint4*>(static_cast<const float*>(g.R) + ro[q]);
        rq[2 * q + 1] = *reinterpret_cast<const uint4*>(static_cast<const float*>(g.R) + ro[q] + 4);
      } else {
        rq[q] = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(g.R) + ro[q]);
      }
    }
  }
  if (!partial) {
    tmem_ld_wait();
  } else {
    // partial + (c4 * 128 + row) * 4 floats; `partial` already points at this row's first chunk
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = 0;
    for (int sp = 0; sp < split_k; ++sp) {
      const float* src = partial + sp * split_stride;
#pragma unroll
      for (int c4 = 0; c4 < 8; ++c4) {
        const float4 f = __ldcg(reinterpret_cast<const float4*>(src + (size_t)c4 * 512));
        r[4 * c4] = __float_as_uint(__uint_as_float(r[4 * c4]) + f.x);
        r[4 * c4 + 1] = __float_as_uint(__uint_as_float(r[4 * c4 + 1]) + f.y);
        r[4 * c4 + 2] = __float_as_uint(__uint_as_float(r[4 * c4 + 2]) + f.z);
        r[4 * c4 + 3] = __float_as_uint(__uint_as_float(r[4 * c4 + 3]) + f.w);
      }
    }
  }
  if (!row_ok) return;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (n + 8 * q >= g.N) break;
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[8 * q + j]) * g.scale;
    if (g.has_bias) {
      const uint32_t w[4] = {bq[q].x, bq[q].y, bq[q].z, bq[q].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[2 * j] += __uint_as_float(w[j] << 16);
        v[2 * j + 1] += __uint_as_float(w[j] & 0xffff0000u);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; j += 2) act2_t<ACT>(v[j], v[j + 1]);
    if (HAS_RES) {
      if (R_WIDE) {
        const uint4 a = rq[2 * q], b = rq[2 * q + 1];
        v[0] += __uint_as_float(a.x); v[1] += __uint_as_float(a.y); v[2] += __uint_as_float(a.z); v[3] += __uint_as_float(a.w);
        v[4] += __uint_as_float(b.x); v[5] += __uint_as_float(b.y); v[6] += __uint_as_float(b.z); v[7] += __uint_as_float(b.w);
      } else {
        const uint32_t w[4] = {rq[q].x, rq[q].y, rq[q].z, rq[q].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[2 * j] += __uint_as_float(w[j] << 16);
          v[2 * j + 1] += __uint_as_float(w[j] & 0xffff0000u);
        }
      }
    }
    if (C_WIDE) {
      float* C = static_cast<float*>(g.C) + co[q];
      *reinterpret_cast<float4*>(C) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<float4*>(C + 4) = make_float4(v[4], v[5], v[6], v[7]);
    } else {
      store16(static_cast<__nv_bfloat16*>(g.C) + co[q], v);
    }
  }
}


// Coalesced vector epilogue for one 32-column chunk of a warp's 32 accumulator rows. Tensor memory
// hands each thread one row; writing rows straight out would touch 32 rows x 16 bytes per store
// instruction. The chunk is therefore turned through a per-warp 4 KB shared-memory tile (16-byte
// units XOR-swizzled by row, conflict-free both ways): afterwards 8 consecutive lanes hold one
// row's 32 columns, so every global access covers 4 rows x 128 (fp32) or 64 (bf16) contiguous bytes.
// Lane l stores rows (l >> 3) + 4 i, i = 0..7, columns 4 (l & 7) .. +3; cbs / rbs are those rows' offsets.
template <int ACT, bool HAS_RES, bool C_WIDE, bool R_WIDE>
__device__ __forceinline__ void epilogue_chunk_coal(const GemmParams& g, uint32_t taddr, const int64_t (&cbs)[8],
                                                    const int64_t (&rbs)[8], uint32_t ok_mask, int n, float* stage, int lane,
                                                    const float* partial, int split_k, size_t split_stride) {
  uint32_t r[32];
  if (!partial) tmem_ld32(taddr, r);
  const int unit = lane & 7, rsub = lane >> 3;
  const int nc = n + unit * 4;
  const bool col_ok = nc < g.N;
  int n1, n0i;
  split2(nc, g.N0, n1, n0i);
  const int64_t c_col = (int64_t)n1 * g.c_s[4] + n0i;
  const int64_t r_col = HAS_RES ? (int64_t)n1 * g.r_s[4] + n0i : 0;
  // operands that do not depend on the accumulator are fetched while the tensor-memory load flies
  float bias4[4] = {0.f, 0.f, 0.f, 0.f};
  if (g.has_bias && col_ok) {
    const uint2 b2 = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.bias) + nc);
    bias4[0] = __uint_as_float(b2.x << 16); bias4[1] = __uint_as_float(b2.x & 0xffff0000u);
    bias4[2] = __uint_as_float(b2.y << 16); bias4[3] = __uint_as_float(b2.y & 0xffff0000u);
  }
  float4 res[HAS_RES ? 8 : 1];
  if (HAS_RES) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      res[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (col_ok && ((ok_mask >> i) & 1u)) {
        if (R_WIDE) {
          res[i] = *reinterpret_cast<const float4*>(static_cast<const float*>(g.R) + rbs[i] + r_col);
        } else {
          const uint2 q = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.R) + rbs[i] + r_col);
          res[i] = make_float4(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u), __uint_as_float(q.y << 16),
                               __uint_as_float(q.y & 0xffff0000u));
        }
      }
    }
  }
  if (!partial) {
    tmem_ld_wait();
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = 0;
    for (int sp = 0; sp < split_k; ++sp) {
      const float* src = partial + sp * split_stride;
#pragma unroll
      for (int c4 = 0; c4 < 8; ++c4) {
        const float4 f = __ldcg(reinterpret_cast<const float4*>(src + (size_t)c4 * 512));
        r[4 * c4] = __float_as_uint(__uint_as_float(r[4 * c4]) + f.x);
        r[4 * c4 + 1] = __float_as_uint(__uint_as_float(r[4 * c4 + 1]) + f.y);
        r[4 * c4 + 2] = __float_as_uint(__uint_as_float(r[4 * c4 + 2]) + f.z);
        r[4 * c4 + 3] = __float_as_uint(__uint_as_float(r[4 * c4 + 3]) + f.w);
      }
    }
  }
  // row `lane` -> shared memory (unit u of row r lives at unit u ^ (r & 7))
#pragma unroll
  for (int u = 0; u < 8; ++u)
    *reinterpret_cast<float4*>(stage + lane * 32 + ((u ^ (lane & 7)) << 2)) =
        make_float4(__uint_as_float(r[4 * u]) * g.scale, __uint_as_float(r[4 * u + 1]) * g.scale,
                    __uint_as_float(r[4 * u + 2]) * g.scale, __uint_as_float(r[4 * u + 3]) * g.scale);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = rsub + 4 * i;
    float4 v = *reinterpret_cast<const float4*>(stage + row * 32 + ((unit ^ (row & 7)) << 2));
    if (!col_ok || !((ok_mask >> i) & 1u)) continue;
    v.x += bias4[0]; v.y += bias4[1]; v.z += bias4[2]; v.w += bias4[3];
    act2_t<ACT>(v.x, v.y);
    act2_t<ACT>(v.z, v.w);
    if (HAS_RES) { v.x += res[i].x; v.y += res[i].y; v.z += res[i].z; v.w += res[i].w; }
    if (C_WIDE) {
      *reinterpret_cast<float4*>(static_cast<float*>(g.C) + cbs[i] + c_col) = v;
    } else {
      *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(g.C) + cbs[i] + c_col) =
          make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
    }
  }
  __syncwarp();   // the tile is reused by the next chunk
}

// The same epilogue for a warp's whole column range [col_begin, col_end) of a tile, software-pipelined
// over its 32-column chunks: the tensor-memory load and the bias of chunk i+1 are in
// flight while chunk i is turned through shared memory and stored (the residual follows as soon as
// chunk i has used its registers), so those latencies overlap the stores instead of preceding them.
template <int ACT, bool HAS_RES, bool C_WIDE, bool R_WIDE>
__device__ __forceinline__ void epilogue_tile_coal(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                   const int64_t (&cbs)[8], const int64_t (&rbs)[8], uint32_t ok_mask,
                                                   float* stage, int lane, float row_scale = 1.f) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const float scale = g.scale * row_scale;   // row_scale: this thread's accumulator row (1 / rms of a split normalisation)
  float* const c_f32 = static_cast<float*>(g.C);
  __nv_bfloat16* const c_b16 = static_cast<__nv_bfloat16*>(g.C);
  int n_chunks = (min(col_end, g.N - n_tile0) - col_begin + 31) >> 5;   // uniform across the warp
  if (n_chunks <= 0) return;
  uint32_t r[32];
  float bias_cur[4], bias_nxt[4] = {0.f, 0.f, 0.f, 0.f};
  float4 res[HAS_RES ? 8 : 1];
  int64_t c_col = 0, c_col_nxt = 0, r_col = 0;
  bool col_ok = false, col_ok_nxt = false;
  // column offsets and bias of the chunk starting at tile column c0
  auto fetch = [&](int c0, float (&bias4)[4], int64_t& ccol, int64_t& rcol, bool& cok) {
    const int nc = n_tile0 + c0 + unit * 4;
    cok = nc < g.N;
    int n1, n0i;
    split2(nc, g.N0, n1, n0i);
    ccol = (int64_t)n1 * g.c_s[4] + n0i;
    if (HAS_RES) rcol = (int64_t)n1 * g.r_s[4] + n0i;
    bias4[0] = bias4[1] = bias4[2] = bias4[3] = 0.f;
    if (g.has_bias && cok) {
      const uint2 b2 = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.bias) + nc);
      bias4[0] = __uint_as_float(b2.x << 16); bias4[1] = __uint_as_float(b2.x & 0xffff0000u);
      bias4[2] = __uint_as_float(b2.y << 16); bias4[3] = __uint_as_float(b2.y & 0xffff0000u);
    }
  };
  // residual of the current chunk (one buffer: the next chunk's loads are issued once this one is consumed)
  auto fetch_res = [&](int64_t rcol, bool cok) {
#pragma unroll
    for (int i = 0; i < (HAS_RES ? 8 : 0); ++i) {
      res[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cok && ((ok_mask >> i) & 1u)) {
        if (R_WIDE) {
          res[i] = *reinterpret_cast<const float4*>(static_cast<const float*>(g.R) + rbs[i] + rcol);
        } else {
          const uint2 q = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.R) + rbs[i] + rcol);
          res[i] = make_float4(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u), __uint_as_float(q.y << 16),
                               __uint_as_float(q.y & 0xffff0000u));
        }
      }
    }
  };
  tmem_ld32(trow + uint32_t(col_begin), r);
  fetch(col_begin, bias_cur, c_col, r_col, col_ok);
  fetch_res(r_col, col_ok);
#pragma unroll 1
  for (int ci = 0; ci < n_chunks; ++ci) {
    tmem_ld_wait();
    // row `lane` -> shared memory (unit u of row r lives at unit u ^ (r & 7))
#pragma unroll
    for (int u = 0; u < 8; ++u)
      sts128(st_row + (uint32_t(u ^ (lane & 7)) << 4), __uint_as_float(r[4 * u]) * scale, __uint_as_float(r[4 * u + 1]) * scale,
             __uint_as_float(r[4 * u + 2]) * scale, __uint_as_float(r[4 * u + 3]) * scale);
    __syncwarp();
    const bool more = ci + 1 < n_chunks;
    int64_t r_col_nxt = 0;
    if (more) {
      const int c0n = col_begin + 32 * (ci + 1);
      tmem_ld32(trow + uint32_t(c0n), r);
      fetch(c0n, bias_nxt, c_col_nxt, r_col_nxt, col_ok_nxt);
    }
    // all eight shared-memory reads first (independent), then the eight stores
    float4 v8[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = rsub + 4 * i;
      v8[i] = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
    }
    // straight-line arithmetic on all eight rows (rows past M and columns past N compute on whatever
    // the accumulator holds and are not stored), then eight predicated stores
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float4& v = v8[i];
      v.x += bias_cur[0]; v.y += bias_cur[1]; v.z += bias_cur[2]; v.w += bias_cur[3];
      act2_t<ACT>(v.x, v.y);
      act2_t<ACT>(v.z, v.w);
      if (HAS_RES) { v.x += res[i].x; v.y += res[i].y; v.z += res[i].z; v.w += res[i].w; }
    }
    const uint32_t live = col_ok ? ok_mask : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (C_WIDE) {
        float4* dst = reinterpret_cast<float4*>(c_f32 + cbs[i] + c_col);
        if ((live >> i) & 1u) *dst = v8[i];
      } else {
        uint2* dst = reinterpret_cast<uint2*>(c_b16 + cbs[i] + c_col);
        const uint2 q = make_uint2(pack_bf16x2(v8[i].x, v8[i].y), pack_bf16x2(v8[i].z, v8[i].w));
        if ((live >> i) & 1u) *dst = q;
      }
    }
    __syncwarp();   // the staging tile is rewritten by the next chunk
    if (more) {
      if (HAS_RES) fetch_res(r_col_nxt, col_ok_nxt);
#pragma unroll
      for (int q = 0; q < 4; ++q) bias_cur[q] = bias_nxt[q];
      c_col = c_col_nxt; col_ok = col_ok_nxt;
    }
  }
}

// The fp32-residual epilogue that also does the first half of an RMS normalisation of its output (the step's output x is
// a residual stream whose only other reader is that normalisation): besides x it writes bf16(x * gain), the A operand of
// the steps behind the normalisation, and the sum of x^2 over this warp's 128 columns of each row, one 128-column slab
// of the row; the readers divide their accumulator rows by the rms they form from the slabs. x is added up and
// rounded exactly as epilogue_tile_coal does it; a tile is 256 columns wide and full (N a multiple of 256), so a warp's
// column range is one slab. row0: the row of the tile that lane 0's first staged row belongs to.
__device__ __forceinline__ void epilogue_tile_resnorm(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                      const int64_t (&cbs)[8], const int64_t (&rbs)[8], uint32_t ok_mask,
                                                      float* stage, int lane, int row0) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const float scale = g.scale;
  float* const c_f32 = static_cast<float*>(g.C);
  __nv_bfloat16* const x_b16 = static_cast<__nv_bfloat16*>(g.nrm_out);
  const __nv_bfloat16* const gain = static_cast<const __nv_bfloat16*>(g.nrm_gamma);
  const int n_chunks = (min(col_end, g.N - n_tile0) - col_begin + 31) >> 5;   // uniform across the warp
  if (n_chunks <= 0) return;
  float ss[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
  for (int ci = 0; ci < n_chunks; ++ci) {
    const int c0 = col_begin + 32 * ci;
    uint32_t r[32];
    tmem_ld32(trow + uint32_t(c0), r);
    const int nc = n_tile0 + c0 + unit * 4;
    const bool col_ok = nc < g.N;
    int n1, n0i;
    split2(nc, g.N0, n1, n0i);
    const int64_t c_col = (int64_t)n1 * g.c_s[4] + n0i, r_col = (int64_t)n1 * g.r_s[4] + n0i;
    float bias4[4] = {0.f, 0.f, 0.f, 0.f}, gain4[4] = {0.f, 0.f, 0.f, 0.f};
    if (col_ok) {
      const uint2 g2 = __ldg(reinterpret_cast<const uint2*>(gain + nc));
      gain4[0] = __uint_as_float(g2.x << 16); gain4[1] = __uint_as_float(g2.x & 0xffff0000u);
      gain4[2] = __uint_as_float(g2.y << 16); gain4[3] = __uint_as_float(g2.y & 0xffff0000u);
      if (g.has_bias) {
        const uint2 b2 = __ldg(reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(g.bias) + nc));
        bias4[0] = __uint_as_float(b2.x << 16); bias4[1] = __uint_as_float(b2.x & 0xffff0000u);
        bias4[2] = __uint_as_float(b2.y << 16); bias4[3] = __uint_as_float(b2.y & 0xffff0000u);
      }
    }
    float4 res[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      res[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (col_ok && ((ok_mask >> i) & 1u)) res[i] = *reinterpret_cast<const float4*>(static_cast<const float*>(g.R) + rbs[i] + r_col);
    }
    tmem_ld_wait();
#pragma unroll
    for (int u = 0; u < 8; ++u)
      sts128(st_row + (uint32_t(u ^ (lane & 7)) << 4), __uint_as_float(r[4 * u]) * scale, __uint_as_float(r[4 * u + 1]) * scale,
             __uint_as_float(r[4 * u + 2]) * scale, __uint_as_float(r[4 * u + 3]) * scale);
    __syncwarp();
    const uint32_t live = col_ok ? ok_mask : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = rsub + 4 * i;
      float4 v = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
      v.x += bias4[0]; v.y += bias4[1]; v.z += bias4[2]; v.w += bias4[3];
      v.x += res[i].x; v.y += res[i].y; v.z += res[i].z; v.w += res[i].w;
      if ((live >> i) & 1u) {
        *reinterpret_cast<float4*>(c_f32 + cbs[i] + c_col) = v;
        *reinterpret_cast<uint2*>(x_b16 + cbs[i] + c_col) = make_uint2(pack_bf16x2(v.x * gain4[0], v.y * gain4[1]), pack_bf16x2(v.z * gain4[2], v.w * gain4[3]));
        ss[i] += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
      }
    }
    __syncwarp();   // the staging tile is rewritten by the next chunk
  }
  // the eight lanes that share a row add up their columns; one of them stores the slab's sum
  const int slab = (n_tile0 + col_begin) >> 7, slabs = g.N >> 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float t = ss[i];
    t += __shfl_xor_sync(0xffffffffu, t, 1);
    t += __shfl_xor_sync(0xffffffffu, t, 2);
    t += __shfl_xor_sync(0xffffffffu, t, 4);
    if (unit == 0 && ((ok_mask >> i) & 1u)) g.nrm_ss[(int64_t)(row0 + rsub + 4 * i) * slabs + slab] = t;
  }
}

// bf16 output without a residual, 64 columns at a time. A thread finishes its own row first (scale, bias, activation,
// rounding), so the staging tile holds 32 rows of 64 bf16 (128 bytes a row, 16-byte units swizzled by the row) and a
// row leaves as ONE 128-byte run (eight lanes x 16 bytes) where the 32-column form above writes two separate 64-byte
// pieces. At the end of a launch every SM stores its last tile at the same moment, and it is the number of write
// requests that reach L2, not their bytes, that sets how long this takes (clock stamps in the 32-column form: ~1200
// cycles a chunk whatever was taken out of it, 13 bytes per cycle and SM for 64-byte pieces against 27 for the
// 128-byte runs of the fp32 outputs). Same arithmetic, in the same order, as the 32-column form.
template <int ACT>
__device__ __forceinline__ void epilogue_tile_coal16(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                     const int64_t (&cbs)[8], uint32_t ok_mask, float* stage, int lane,
                                                     float row_scale = 1.f) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const float scale = g.scale * row_scale;
  __nv_bfloat16* const c_b16 = static_cast<__nv_bfloat16*>(g.C);
  const __nv_bfloat16* const bias = static_cast<const __nv_bfloat16*>(g.bias);
  const int n_chunks = (min(col_end, g.N - n_tile0) - col_begin + 63) >> 6;   // uniform across the warp
  if (n_chunks <= 0) return;
  uint32_t r[32];
  tmem_ld32(trow + uint32_t(col_begin), r);
#pragma unroll 1
  for (int ci = 0; ci < n_chunks; ++ci) {
    const int c0 = col_begin + 64 * ci;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      // bias of these 32 columns, the same for every row of the warp: four 16-byte loads that every lane shares
      uint4 b4[4];
      const int nb = n_tile0 + c0 + 32 * h;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        b4[k] = (g.has_bias && nb + 8 * k < g.N) ? __ldg(reinterpret_cast<const uint4*>(bias + nb + 8 * k)) : make_uint4(0u, 0u, 0u, 0u);
      tmem_ld_wait();
      float v[32];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t w[4] = {b4[k].x, b4[k].y, b4[k].z, b4[k].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          v[8 * k + 2 * q] = __uint_as_float(r[8 * k + 2 * q]) * scale + __uint_as_float(w[q] << 16);
          v[8 * k + 2 * q + 1] = __uint_as_float(r[8 * k + 2 * q + 1]) * scale + __uint_as_float(w[q] & 0xffff0000u);
        }
      }
      // the next 32 columns are on their way while these are finished (the accumulator is 64 ci + 64 columns wide at least)
      if (h == 0 || ci + 1 < n_chunks) tmem_ld32(trow + uint32_t(c0 + 32 * (h + 1)), r);
#pragma unroll
      for (int k = 0; k < 16; ++k) act2_t<ACT>(v[2 * k], v[2 * k + 1]);
#pragma unroll
      for (int k = 0; k < 4; ++k)   // unit 4 h + k of row `lane` lives at unit (4 h + k) ^ (lane & 7)
        sts128(st_row + (uint32_t((4 * h + k) ^ (lane & 7)) << 4), __uint_as_float(pack_bf16x2(v[8 * k], v[8 * k + 1])),
               __uint_as_float(pack_bf16x2(v[8 * k + 2], v[8 * k + 3])), __uint_as_float(pack_bf16x2(v[8 * k + 4], v[8 * k + 5])),
               __uint_as_float(pack_bf16x2(v[8 * k + 6], v[8 * k + 7])));
    }
    __syncwarp();
    // lane (rsub, unit): rows rsub + 4 i, columns 8 unit .. 8 unit + 7 of the chunk
    const int nc = n_tile0 + c0 + unit * 8;
    int n1, n0i;
    split2(nc, g.N0, n1, n0i);
    const int64_t c_col = (int64_t)n1 * g.c_s[4] + n0i;
    const uint32_t live = nc < g.N ? ok_mask : 0u;
    float4 v8[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = rsub + 4 * i;
      v8[i] = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint4* dst = reinterpret_cast<uint4*>(c_b16 + cbs[i] + c_col);
      if ((live >> i) & 1u)
        *dst = make_uint4(__float_as_uint(v8[i].x), __float_as_uint(v8[i].y), __float_as_uint(v8[i].z), __float_as_uint(v8[i].w));
    }
    __syncwarp();   // the staging tile is rewritten by the next chunk
  }
}

// General epilogue for one 8-column group: any strides, any tails, any storage width.
__device__ __noinline__ void epilogue_group_any(const GemmParams& g, uint32_t taddr, bool row_ok, int64_t cb, int64_t rb,
                                                int n) {
  uint32_t r[8];
  tmem_ld8(taddr, r);
  tmem_ld_wait();
  if (!row_ok) return;
  const bool c_wide = g.c_f32 != 0, r_wide = g.r_f32 != 0;
#pragma unroll 1
  for (int j = 0; j < 8; ++j) {
    if (n + j >= g.N) break;
    float v = __uint_as_float(r[0]) * g.scale;
#pragma unroll
    for (int q = 1; q < 8; ++q) v = j == q ? __uint_as_float(r[q]) * g.scale : v;
    if (g.has_bias) v += to_f(static_cast<const __nv_bfloat16*>(g.bias)[n + j]);
    v = g.act == ACT_GELU_ERF ? gelu_erf_fast(v) : (g.act == ACT_GELU_TANH ? gelu_tanh(v) : v);
    if (g.has_res) {
      const int64_t rj = rb + split_off(n + j, g.N0, g.r_s[4], g.r_s[5]);
      v += r_wide ? static_cast<const float*>(g.R)[rj] : to_f(static_cast<const __nv_bfloat16*>(g.R)[rj]);
    }
    const int64_t cj = cb + split_off(n + j, g.N0, g.c_s[4], g.c_s[5]);
    if (c_wide) static_cast<float*>(g.C)[cj] = v;
    else static_cast<__nv_bfloat16*>(g.C)[cj] = __float2bfloat16_rn(v);
  }
}

// General epilogue for outputs whose rows are not 16-byte aligned (an odd N, e.g. a vocabulary size)
// but whose n index is contiguous and unsplit: the same shared-memory turn as the vector variants, then
// scalar loads and stores, so that the lanes of a warp still cover runs of consecutive columns instead
// of one row each. Flags are read at run time (this is the rare path).
__device__ __noinline__ void epilogue_tile_scalar(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                  int64_t cbz, int64_t rbz, int m_base, float* stage, int lane) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const bool c_wide = g.c_f32 != 0, r_wide = g.r_f32 != 0;
  const float scale = g.scale;
#pragma unroll 1
  for (int c0 = col_begin; c0 < col_end; c0 += 32) {
    if (n_tile0 + c0 >= g.N) break;   // uniform across the warp
    uint32_t r[32];
    tmem_ld32(trow + uint32_t(c0), r);
    tmem_ld_wait();
#pragma unroll
    for (int u = 0; u < 8; ++u)
      sts128(st_row + (uint32_t(u ^ (lane & 7)) << 4), __uint_as_float(r[4 * u]) * scale, __uint_as_float(r[4 * u + 1]) * scale,
             __uint_as_float(r[4 * u + 2]) * scale, __uint_as_float(r[4 * u + 3]) * scale);
    __syncwarp();
    const int nc = n_tile0 + c0 + unit * 4;
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
      const int row = rsub + 4 * i, m = m_base + row;
      if (m >= g.M) break;            // rows only grow with i
      const float4 q = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
      const float v4[4] = {q.x, q.y, q.z, q.w};
      const int64_t cb = cbz + split_off(m, g.M0, g.c_s[2], g.c_s[3]);
      const int64_t rb = g.has_res ? rbz + split_off(m, g.M0, g.r_s[2], g.r_s[3]) : 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int n = nc + e;
        if (n >= g.N) break;
        float v = v4[e];
        if (g.has_bias) v += to_f(static_cast<const __nv_bfloat16*>(g.bias)[n]);
        v = g.act == ACT_GELU_ERF ? gelu_erf_fast(v) : (g.act == ACT_GELU_TANH ? gelu_tanh(v) : v);
        if (g.has_res) v += r_wide ? static_cast<const float*>(g.R)[rb + n] : to_f(static_cast<const __nv_bfloat16*>(g.R)[rb + n]);
        if (c_wide) static_cast<float*>(g.C)[cb + n] = v;
        else static_cast<__nv_bfloat16*>(g.C)[cb + n] = __float2bfloat16_rn(v);
      }
    }
    __syncwarp();   // the staging tile is rewritten by the next chunk
  }
}

// Epilogue variants (template parameter of the kernel)
enum EpiKind { EPI_ANY = 0, EPI_PLAIN = 1, EPI_PLAIN_WIDE = 2, EPI_RES = 3, EPI_RES_WIDE = 4, EPI_GELU_ERF = 5, EPI_GELU_TANH = 6,
               EPI_SWIGLU = 7 /* CTA-pair kernel only */, EPI_ROPE = 8 /* CTA-pair kernel only: plain, with the rotary embedding for groups that ask */,
               EPI_RES_WIDE_NRM = 9 /* CTA-pair kernel only: fp32 residual in / out, plus the first half of an RMS normalisation of the output */ };

template <int EPI>
__device__ __forceinline__ void epilogue_chunk_c(const GemmParams& g, uint32_t taddr, const int64_t (&cbs)[8], const int64_t (&rbs)[8],
                                                 uint32_t ok_mask, int n, float* stage, int lane, const float* partial = nullptr,
                                                 int sk = 1, size_t ss = 0) {
  if (EPI == EPI_PLAIN) epilogue_chunk_coal<ACT_NONE, false, false, false>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
  else if (EPI == EPI_PLAIN_WIDE) epilogue_chunk_coal<ACT_NONE, false, true, false>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
  else if (EPI == EPI_RES) epilogue_chunk_coal<ACT_NONE, true, false, false>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
  else if (EPI == EPI_RES_WIDE) epilogue_chunk_coal<ACT_NONE, true, true, true>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
  else if (EPI == EPI_GELU_ERF) epilogue_chunk_coal<ACT_GELU_ERF, false, false, false>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
  else if (EPI == EPI_GELU_TANH) epilogue_chunk_coal<ACT_GELU_TANH, false, false, false>(g, taddr, cbs, rbs, ok_mask, n, stage, lane, partial, sk, ss);
}

template <int EPI>
__device__ __forceinline__ void epilogue_tile_c(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                const int64_t (&cbs)[8], const int64_t (&rbs)[8], uint32_t ok_mask, float* stage,
                                                int lane, float row_scale = 1.f) {
  // bf16 outputs without a residual leave in 128-byte runs when the warp's columns come in sixty-fours
  const bool wide_runs = ((col_end - col_begin) & 63) == 0;
  if (EPI == EPI_PLAIN && wide_runs) epilogue_tile_coal16<ACT_NONE>(g, trow, col_begin, col_end, n_tile0, cbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_GELU_ERF && wide_runs) epilogue_tile_coal16<ACT_GELU_ERF>(g, trow, col_begin, col_end, n_tile0, cbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_GELU_TANH && wide_runs) epilogue_tile_coal16<ACT_GELU_TANH>(g, trow, col_begin, col_end, n_tile0, cbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_PLAIN) epilogue_tile_coal<ACT_NONE, false, false, false>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_PLAIN_WIDE) epilogue_tile_coal<ACT_NONE, false, true, false>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_RES) epilogue_tile_coal<ACT_NONE, true, false, false>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_RES_WIDE) epilogue_tile_coal<ACT_NONE, true, true, true>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_GELU_ERF) epilogue_tile_coal<ACT_GELU_ERF, false, false, false>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
  else if (EPI == EPI_GELU_TANH) epilogue_tile_coal<ACT_GELU_TANH, false, false, false>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
}

template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& g, uint32_t taddr, bool row_ok, int64_t cb, int64_t rb, int n,
                                               const float* partial = nullptr, int sk = 1, size_t ss = 0) {
  if (EPI == EPI_PLAIN) epilogue_chunk_vec<ACT_NONE, false, false, false>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else if (EPI == EPI_PLAIN_WIDE) epilogue_chunk_vec<ACT_NONE, false, true, false>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else if (EPI == EPI_RES) epilogue_chunk_vec<ACT_NONE, true, false, false>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else if (EPI == EPI_RES_WIDE) epilogue_chunk_vec<ACT_NONE, true, true, true>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else if (EPI == EPI_GELU_ERF) epilogue_chunk_vec<ACT_GELU_ERF, false, false, false>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else if (EPI == EPI_GELU_TANH) epilogue_chunk_vec<ACT_GELU_TANH, false, false, false>(g, taddr, row_ok, cb, rb, n, partial, sk, ss);
  else {
#pragma unroll 1
    for (int q = 0; q < 4; ++q) {
      if (n + 8 * q >= g.N) break;
      epilogue_group_any(g, taddr + 8 * q, row_ok, cb, rb, n + 8 * q);
    }
  }
}

template <int EPI, bool SPLIT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
               const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte-swizzle atoms want 1024-byte alignment
  const int bn = p.cfg.bn, stages = p.cfg.stages;
  const uint32_t b_tile_bytes = uint32_t(bn) * BK * 2;
  const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
  const uint32_t bars = base + uint32_t(stages) * stage_bytes;  // 8-byte barriers after the tiles
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (stages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * stages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * stages + 2 + a); };
  const uint32_t tmem_slot = bars + 8u * (2 * stages + 4);
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  volatile uint32_t* abort_flag = tmem_slot_ptr + 1;
  const uint32_t stage_base = (tmem_slot + 16u + 15u) & ~15u;   // 8 warps x 4 KB epilogue staging tiles

  pdl_launch_dependents();  // the next step may start its prologue now
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_cols = uint32_t(2 * bn);  // 128, 256 or 512: a power of two >= 32

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), kEpiWarps); }
    *abort_flag = 0;
    abort_flag[2] = 0;   // split-K epilogue: set when a warp's accumulator wait gave up
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    // One lane per 64-wide box of a stage: lanes 0-1 the A boxes, lanes 2-5 the B boxes (a K-major
    // operand is one box, an MN-major one is a box per 64 rows). The lanes run in lockstep on the
    // same barriers, so the per-tile coordinate set-up (divisions, selects) costs one box's worth
    // and the per-k-step loop is a wait, one TMA and three adds. A single thread issuing every
    // box was the slowest part of a short tile (about 600 cycles per k-step, 3000 per tile).
    const bool is_a = lane < 2;
    const int ch = is_a ? lane : lane - 2;
    // boxes per tile and rows per box: an MN-major operand comes in boxes of 64 rows, a K-major A in one box, a
    // K-major B in boxes of b_box_rows rows (one, or two when the tensor map was cut for a CTA pair)
    const int box_rows = (is_a ? p.cfg.a_mn_major : p.cfg.b_mn_major) ? 64 : (is_a ? BM : p.cfg.b_box_rows);
    const int n_box = (is_a ? BM : bn) / box_rows;
    if (lane < 6 && ch < n_box) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true, in_flight = false;
      const uint32_t box_off = (is_a ? 0u : kATileBytes) + uint32_t(ch) * uint32_t(box_rows) * 128u;
      const int x_r0 = is_a ? p.cfg.a_r0 : p.cfg.b_r0, x_b0 = is_a ? p.cfg.a_b0 : p.cfg.b_b0;
      const int x_k0 = is_a ? p.cfg.a_k0 : p.cfg.b_k0;
      int sel[5];
#pragma unroll
      for (int d = 0; d < 5; ++d) sel[d] = is_a ? p.cfg.a_sel[d] : p.cfg.b_sel[d];
      // which coordinate slots carry the running k split (the rest stay fixed over a tile)
      int kd0 = 0, kd1 = -1;
#pragma unroll
      for (int d = 0; d < 5; ++d) {
        if (sel[d] == 0) kd0 = d;
        if (sel[d] == 1) kd1 = d;
      }
      // k in one tensor-map dim (0 for a K-major operand, 1 or 2 for an MN-major one): running sums only
      const bool k_simple = kd1 < 0 && kd0 < 3;
      const int i0 = kd0 == 0 ? BK : 0, i1 = kd0 == 1 ? BK : 0, i2 = kd0 == 2 ? BK : 0;
      uint32_t dst = base + box_off, fb = full_bar(0), eb = empty_bar(0);   // the running stage
      // The previous step's outputs are this step's operands, except for weights: a constant B is loaded
      // while the previous step is still finishing (its bytes may land before lane 0 posts the expected
      // count; the barrier's pending arrival keeps the phase open until then).
      const bool b_free = p.g.b_const && (p.n_group < 2 || p.gx[0].b_const) && (p.n_group < 3 || p.gx[1].b_const);
      // A tile's coordinates are index arithmetic only (divisions and selects, ~1 us on this one warp): the first tile's are
      // ready before the wait for the previous step, every later tile's while its predecessor's loads are in flight
      int c[5], ksteps = 0, k_begin = 0;
      const CUtensorMap* map = &map_a;
      auto prep = [&](int item) {
        int tile, sp, k_count;
        decode_item<SPLIT>(p, item, tile, sp, k_begin, k_count);
        int grp, bz, mt, nt;
        decode_tile(p, tile, grp, bz, mt, nt);
        ksteps = k_count >= 0 ? k_count : k_steps_of(p, mt);
        int r1, r0, b1, b0;
        split2((is_a ? mt * BM : nt * bn) + ch * box_rows, x_r0, r1, r0);
        split2(bz, x_b0, b1, b0);
        fill_coords(sel, 5, 0, 0, r0, r1, b0, b1, c);
        map = is_a ? &map_a : (grp == 0 ? &map_b : (grp == 1 ? &map_b1 : &map_b2));
      };
      int item = blockIdx.x;
      if (item < p.num_tiles) prep(item);
      if (is_a || !b_free) pdl_wait();
      for (; ok && item < p.num_tiles; item += gridDim.x, (item < p.num_tiles ? prep(item) : (void)0)) {
        if (k_simple) {
          const int kc = k_begin * BK;
          c[0] += i0 ? kc : 0; c[1] += i1 ? kc : 0; c[2] += i2 ? kc : 0;
          for (int ks = 0; ks < ksteps; ++ks) {
            if (!mbar_wait(eb, ph ^ 1u)) { ok = false; break; }
            if (lane == 0) mbar_expect_tx(fb, stage_bytes);
            tma_load(dst, map, fb, c[0], c[1], c[2], c[3], c[4]);
            in_flight = true;
            c[0] += i0; c[1] += i1; c[2] += i2;
            dst += stage_bytes; fb += 8u; eb += 8u;
            if (++s == stages) { s = 0; ph ^= 1u; dst = base + box_off; fb = full_bar(0); eb = empty_bar(0); }
          }
          continue;
        }
        int k0, k1;  // running two-level split of the k index
        split2(k_begin * BK, x_k0, k1, k0);
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(eb, ph ^ 1u)) { ok = false; break; }
          if (lane == 0) mbar_expect_tx(fb, stage_bytes);
          int q[5];
#pragma unroll
          for (int d = 0; d < 5; ++d) q[d] = c[d] + (d == kd0 ? k0 : 0) + (d == kd1 ? k1 : 0);
          tma_load(dst, map, fb, q[0], q[1], q[2], q[3], q[4]);
          in_flight = true;
          k0 += BK; if (k0 >= x_k0) { k0 = 0; ++k1; }
          dst += stage_bytes; fb += 8u; eb += 8u;
          if (++s == stages) { s = 0; ph ^= 1u; dst = base + box_off; fb = full_bar(0); eb = empty_bar(0); }
        }
      }
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x1u);
        *abort_flag = 1;
        // let the loads already issued land before this CTA's shared memory is given up: the most
        // recent fill of every stage this lane wrote (stages before s are in phase ph, the rest in ph ^ 1)
        if (in_flight)
          for (int j = 0; j < stages; ++j) mbar_wait(full_bar(j), j < s ? ph : ph ^ 1u);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = make_idesc(bn, p.cfg.a_mn_major, p.cfg.b_mn_major);
      // 16-byte units between the four 16-deep k slices of a stage: 32 bytes along a K-major row,
      // 2048 bytes (16 k-rows of 128 bytes) in an MN-major tile
      const uint32_t a_step = p.cfg.a_mn_major ? 128u : 2u, b_step = p.cfg.b_mn_major ? 128u : 2u;
      const uint64_t ad_first = make_desc(base, p.cfg.a_mn_major), bd_first = make_desc(base + kATileBytes, p.cfg.b_mn_major);
      const uint32_t a_hi = uint32_t(ad_first >> 32), b_hi = uint32_t(bd_first >> 32);
      const uint32_t a_lo0 = uint32_t(ad_first), b_lo0 = uint32_t(bd_first), stage16 = stage_bytes >> 4;
      // the running stage: descriptor low words (the address field never carries out of its 14 bits,
      // shared memory being smaller than 256 KB) and barrier addresses
      uint32_t a_lo = a_lo0, b_lo = b_lo0, fb = full_bar(0), eb = empty_bar(0);
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < p.num_tiles; item += gridDim.x) {
        int tile, sp, k_begin, k_count;
        decode_item<SPLIT>(p, item, tile, sp, k_begin, k_count);
        int grp, bz, mt, nt;
        decode_tile(p, tile, grp, bz, mt, nt);
        const int ksteps = k_count >= 0 ? k_count : k_steps_of(p, mt);
        if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_c = tmem_base + uint32_t(acc * bn);
        uint32_t accum = 0u;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(fb, ph)) { ok = false; break; }
          tc_fence_after();
          umma_bf16_lohi(tmem_c, a_lo, a_hi, b_lo, b_hi, idesc, accum);
          umma_bf16_lohi(tmem_c, a_lo + a_step, a_hi, b_lo + b_step, b_hi, idesc, 1u);
          umma_bf16_lohi(tmem_c, a_lo + 2u * a_step, a_hi, b_lo + 2u * b_step, b_hi, idesc, 1u);
          umma_bf16_lohi(tmem_c, a_lo + 3u * a_step, a_hi, b_lo + 3u * b_step, b_hi, idesc, 1u);
          umma_commit(eb);  // the stage is free once these MMAs have read it
          accum = 1u;
          a_lo += stage16; b_lo += stage16; fb += 8u; eb += 8u;
          if (++s == stages) { s = 0; ph ^= 1u; a_lo = a_lo0; b_lo = b_lo0; fb = full_bar(0); eb = empty_bar(0); }
        }
        if (ok) umma_commit(tfull_bar(acc));  // accumulator complete
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x2u);
        *abort_flag = 1;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..9) ----------------
    // Warp w reads tensor-memory lanes 32*(w%4)..+31 (one accumulator row per thread); the two
    // warps that share a lane quarter split the tile's columns between them.
    const int lane_base = (warp & 3) * 32;
    const int half = (warp - 2) >> 2;
    float* stage = reinterpret_cast<float*>(smem_raw + (stage_base - raw)) + (warp - 2) * 1024;
    const int col_begin = half * (bn / 2), col_end = col_begin + bn / 2;
    int acc = 0;
    uint32_t acc_ph = 0;
    bool ok = true;
    bool waited = false;
    for (int item = blockIdx.x; ok && item < p.num_tiles; item += gridDim.x) {
      int tile, sp, k_begin, k_count;
      decode_item<SPLIT>(p, item, tile, sp, k_begin, k_count);
      int grp, bz, mt, nt;
      decode_tile(p, tile, grp, bz, mt, nt);
      const GemmParams& g = grp == 0 ? p.g : p.gx[grp - 1];
      const int m = mt * BM + lane_base + lane;
      const bool row_ok = m < g.M;
      const int64_t cb = split_off(bz, g.B0, g.c_s[0], g.c_s[1]) + (row_ok ? split_off(m, g.M0, g.c_s[2], g.c_s[3]) : 0);
      const int64_t rb = g.has_res ? split_off(bz, g.B0, g.r_s[0], g.r_s[1]) + (row_ok ? split_off(m, g.M0, g.r_s[2], g.r_s[3]) : 0) : 0;
      const int n_tile0 = nt * bn;
      // vector variants: offsets of the 8 rows this lane stores after the shared-memory turn
      int64_t cbs[8], rbs[8];
      uint32_t ok_mask = 0;
      if (EPI != EPI_ANY) {
        const int64_t cbz = split_off(bz, g.B0, g.c_s[0], g.c_s[1]);
        const int64_t rbz = g.has_res ? split_off(bz, g.B0, g.r_s[0], g.r_s[1]) : 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int mi = mt * BM + lane_base + (lane >> 3) + 4 * i;
          const bool live = mi < g.M;
          ok_mask |= live ? (1u << i) : 0u;
          cbs[i] = cbz + (live ? split_off(mi, g.M0, g.c_s[2], g.c_s[3]) : 0);
          rbs[i] = g.has_res ? rbz + (live ? split_off(mi, g.M0, g.r_s[2], g.r_s[3]) : 0) : 0;
        }
      }
      // the first tile's row and column offsets above are index arithmetic: done before the wait
      if (!waited) { pdl_wait(); waited = true; }   // before any global read (bias, residual) or write (C)
      bool got = mbar_wait_warp(tfull_bar(acc), acc_ph);
      if (SPLIT) {
        // the eight epilogue warps meet at named barriers below: either all of them go on or none does
        if (!got && lane == 0) abort_flag[2] = 1;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        got = abort_flag[2] == 0;
      }
      if (!got) { ok = false; break; }
      tc_fence_after();
      const uint32_t trow = tmem_base + (uint32_t(lane_base) << 16) + uint32_t(acc * bn);
      if (!SPLIT) {
        if (EPI == EPI_ANY && p.scalar_turn) {
          epilogue_tile_scalar(g, trow, col_begin, col_end, n_tile0, split_off(bz, g.B0, g.c_s[0], g.c_s[1]),
                               g.has_res ? split_off(bz, g.B0, g.r_s[0], g.r_s[1]) : 0, mt * BM + lane_base, stage, lane);
        } else if (EPI == EPI_ANY) {
#pragma unroll 1
          for (int c0 = col_begin; c0 < col_end; c0 += 32) {
            if (n_tile0 + c0 >= g.N) break;  // whole chunk out of range (uniform across the warp)
            epilogue_chunk<EPI>(g, trow + uint32_t(c0), row_ok, cb, rb, n_tile0 + c0);
          }
        } else {
          epilogue_tile_c<EPI>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));
      } else {
        // ---- split-K: park this CTA's partial tile, the last CTA to arrive adds them up ----
        const size_t tile_floats = size_t(BM) * bn;
        float* mine = p.partial + (size_t(tile) * p.split_k + sp) * tile_floats + size_t(lane_base + lane) * 4;
#pragma unroll 1
        for (int c0 = col_begin; c0 < col_end; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(trow + uint32_t(c0), r);
          tmem_ld_wait();
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4)
            __stcg(reinterpret_cast<float4*>(mine + size_t(c0 / 4 + c4) * 512),
                   make_float4(__uint_as_float(r[4 * c4]), __uint_as_float(r[4 * c4 + 1]), __uint_as_float(r[4 * c4 + 2]),
                               __uint_as_float(r[4 * c4 + 3])));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));   // the accumulator is free again
        __threadfence();
        asm volatile("bar.sync 1, 256;" ::: "memory");      // all eight epilogue warps have stored
        if (warp == 2 && lane == 0) {
          const uint32_t prev = atomicAdd(p.status + 8 + tile, 1u);
          *reinterpret_cast<volatile uint32_t*>(abort_flag + 1) = prev;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const bool last = *reinterpret_cast<volatile uint32_t*>(abort_flag + 1) == uint32_t(p.split_k - 1);
        if (last) {
          __threadfence();
          const float* base_row = p.partial + size_t(tile) * p.split_k * tile_floats + size_t(lane_base + lane) * 4;
#pragma unroll 1
          for (int c0 = col_begin; c0 < col_end; c0 += 32) {
            if (n_tile0 + c0 >= g.N) break;
            epilogue_chunk_c<EPI>(g, 0u, cbs, rbs, ok_mask, n_tile0 + c0, stage, lane, base_row + size_t(c0 / 4) * 512, p.split_k, tile_floats);
          }
          if (warp == 2 && lane == 0) p.status[8 + tile] = 0;   // ready for the next launch
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");      // the exchange word is reused by the next item
      }
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    if (!ok && lane == 0) {
      if (!*abort_flag) atomicOr(p.status, 0x4u);
      *abort_flag = 1;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ---- cluster split-K: short-and-wide GEMMs (few output tiles, e.g. 128 tokens) -----------------------
// With one row of output tiles a launch of the persistent kernel occupies a handful of SMs, and every
// one of them walks the whole K range at the tensor core's fixed ~128 cycles per 128 x N x 16
// instruction. Here a thread-block cluster of `split_k` CTAs shares one output tile: CTA r runs the
// k-steps [r * kps, (r + 1) * kps) into its own tensor-memory accumulator, then the cluster
// reduce-scatters the fp32 partials through distributed shared memory: every CTA lays its partial
// tile out in its own shared memory (over the drained pipeline stages) and sends rows
// [d * 128 / split_k, ...) to CTA d with one bulk copy that completes on d's receive barrier; CTA d
// sums the split_k slices in rank order (deterministic) and runs the epilogue for its rows.
// No global scratch, no atomics. Warp roles as in the persistent kernel. Every thread of the cluster
// passes both cluster barriers on every path (the bounded mbarrier waits only skip work), so a
// failed wait cannot leave a peer waiting; the second barrier also keeps a CTA's shared memory alive
// until its outgoing copies have landed.
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  return remote;
}
// shared memory of this CTA -> shared memory of a CTA of the cluster, completing on that CTA's mbarrier
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t bar_cluster) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_cluster), "r"(src_cta), "r"(bytes), "r"(bar_cluster) : "memory");
}

// What the last phase needs of a GemmParams, read into registers once (before the wait for the peers'
// slices, so that the parameter reads overlap it).
struct FinalCtx {
  void* C;
  const void* R;
  const __nv_bfloat16* bias;
  int64_t cs4, rs4;
  int N0;
  float scale;
};

template <int ACT, bool HAS_RES, bool C_WIDE, bool R_WIDE>
__device__ __forceinline__ void final_store4(const FinalCtx& f, float4 v, int64_t cb, int64_t rb, int nc) {
  int n1, n0i;
  split2(nc, f.N0, n1, n0i);
  v.x *= f.scale; v.y *= f.scale; v.z *= f.scale; v.w *= f.scale;
  if (f.bias) {
    const uint2 b2 = *reinterpret_cast<const uint2*>(f.bias + nc);
    v.x += __uint_as_float(b2.x << 16); v.y += __uint_as_float(b2.x & 0xffff0000u);
    v.z += __uint_as_float(b2.y << 16); v.w += __uint_as_float(b2.y & 0xffff0000u);
  }
  act2_t<ACT>(v.x, v.y);
  act2_t<ACT>(v.z, v.w);
  if (HAS_RES) {
    const int64_t ro = rb + (int64_t)n1 * f.rs4 + n0i;
    if (R_WIDE) {
      const float4 q = *reinterpret_cast<const float4*>(static_cast<const float*>(f.R) + ro);
      v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
    } else {
      const uint2 q = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(f.R) + ro);
      v.x += __uint_as_float(q.x << 16); v.y += __uint_as_float(q.x & 0xffff0000u);
      v.z += __uint_as_float(q.y << 16); v.w += __uint_as_float(q.y & 0xffff0000u);
    }
  }
  const int64_t co = cb + (int64_t)n1 * f.cs4 + n0i;
  if (C_WIDE) *reinterpret_cast<float4*>(static_cast<float*>(f.C) + co) = v;
  else *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(f.C) + co) = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
}

template <int EPI>
__device__ __forceinline__ void final_store4_c(const FinalCtx& f, float4 v, int64_t cb, int64_t rb, int nc) {
  if (EPI == EPI_PLAIN) final_store4<ACT_NONE, false, false, false>(f, v, cb, rb, nc);
  else if (EPI == EPI_PLAIN_WIDE) final_store4<ACT_NONE, false, true, false>(f, v, cb, rb, nc);
  else if (EPI == EPI_RES) final_store4<ACT_NONE, true, false, false>(f, v, cb, rb, nc);
  else if (EPI == EPI_RES_WIDE) final_store4<ACT_NONE, true, true, true>(f, v, cb, rb, nc);
  else if (EPI == EPI_GELU_ERF) final_store4<ACT_GELU_ERF, false, false, false>(f, v, cb, rb, nc);
  else final_store4<ACT_GELU_TANH, false, false, false>(f, v, cb, rb, nc);
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_cluster_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                       const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const int bn = p.cfg.bn, stages = p.cfg.stages, sk = p.split_k;
  const uint32_t stage_bytes = kATileBytes + uint32_t(bn) * BK * 2;
  const uint32_t recv = base + uint32_t(stages) * stage_bytes;       // [split][128 / sk rows][bn] fp32, 16-byte units swizzled by row
  const uint32_t bars = recv + uint32_t(BM) * uint32_t(bn) * 4u;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (stages + s); };
  const uint32_t tfull = bars + 8u * (2 * stages);
  const uint32_t recv_bar = tfull + 8u;
  const uint32_t tmem_slot = recv_bar + 8u;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  volatile uint32_t* abort_flag = tmem_slot_ptr + 1;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_cols = uint32_t(bn < 32 ? 32 : bn);
  const int sp = (int)cluster_rank();
  const int tile = int(blockIdx.x) / sk;
  const int total_ksteps = (p.g.K + BK - 1) / BK;
  const int k_begin = sp * p.ksteps_per_split;
  const int ksteps = min(p.ksteps_per_split, total_ksteps - k_begin);   // >= 1 by the host's choice of sk
  int grp, bz, mt, nt;
  decode_tile(p, tile, grp, bz, mt, nt);

  // The producer warp needs the barriers, not the tensor-memory address: it initialises them, arrives on a named
  // barrier and goes on to its loads while warp 1 allocates tensor memory; everyone else waits for both.
  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
      mbar_init(tfull, 1);
      mbar_init(recv_bar, 1);
      *abort_flag = 0;
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      mbar_expect_tx(recv_bar, uint32_t(BM) * uint32_t(bn) * 4u);   // split_k slices of 128 / split_k rows
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
    }
    __syncwarp();
    __threadfence_block();
    asm volatile("bar.arrive 2, 320;" ::: "memory");
  } else {
    if (warp == 1) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    asm volatile("bar.sync 2, 320;" ::: "memory");
    tc_fence_after();
  }
  const uint32_t tmem_base = *tmem_slot_ptr;   // (not meaningful in warp 0, which does not use it)
  cluster_arrive();   // "this CTA runs": peers may write into its receive buffer after the matching wait

  if (warp == 0) {
    // ---------------- TMA producer: one lane per 64-wide box, as in the persistent kernel ----------------
    const bool is_a = lane < 2;
    const int ch = is_a ? lane : lane - 2;
    // boxes per tile and rows per box: an MN-major operand comes in boxes of 64 rows, a K-major A in one box, a
    // K-major B in boxes of b_box_rows rows (one, or two when the tensor map was cut for a CTA pair)
    const int box_rows = (is_a ? p.cfg.a_mn_major : p.cfg.b_mn_major) ? 64 : (is_a ? BM : p.cfg.b_box_rows);
    const int n_box = (is_a ? BM : bn) / box_rows;
    if (lane < 6 && ch < n_box) {
      const uint32_t box_off = (is_a ? 0u : kATileBytes) + uint32_t(ch) * uint32_t(box_rows) * 128u;
      const int x_r0 = is_a ? p.cfg.a_r0 : p.cfg.b_r0, x_b0 = is_a ? p.cfg.a_b0 : p.cfg.b_b0;
      const int x_k0 = is_a ? p.cfg.a_k0 : p.cfg.b_k0;
      int sel[5];
#pragma unroll
      for (int d = 0; d < 5; ++d) sel[d] = is_a ? p.cfg.a_sel[d] : p.cfg.b_sel[d];
      int kd0 = 0, kd1 = -1;
#pragma unroll
      for (int d = 0; d < 5; ++d) {
        if (sel[d] == 0) kd0 = d;
        if (sel[d] == 1) kd1 = d;
      }
      int c[5];
      {
        int r1, r0, b1, b0;
        split2((is_a ? mt * BM : nt * bn) + ch * box_rows, x_r0, r1, r0);
        split2(bz, x_b0, b1, b0);
        fill_coords(sel, 5, 0, 0, r0, r1, b0, b1, c);
      }
      const CUtensorMap* map = is_a ? &map_a : (grp == 0 ? &map_b : (grp == 1 ? &map_b1 : &map_b2));
      int k0, k1;
      split2(k_begin * BK, x_k0, k1, k0);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      // weights do not wait for the previous step (see the persistent kernel's producer)
      const bool b_free = p.g.b_const && (p.n_group < 2 || p.gx[0].b_const) && (p.n_group < 3 || p.gx[1].b_const);
      if (is_a || !b_free) pdl_wait();
      if (kd1 < 0 && kd0 < 3) {
        const int i0 = kd0 == 0 ? BK : 0, i1 = kd0 == 1 ? BK : 0, i2 = kd0 == 2 ? BK : 0;
        c[0] += i0 ? k0 : 0; c[1] += i1 ? k0 : 0; c[2] += i2 ? k0 : 0;
        uint32_t dst = base + box_off, fb = full_bar(0), eb = empty_bar(0);
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(eb, ph ^ 1u)) { ok = false; break; }
          if (lane == 0) mbar_expect_tx(fb, stage_bytes);
          tma_load(dst, map, fb, c[0], c[1], c[2], c[3], c[4]);
          c[0] += i0; c[1] += i1; c[2] += i2;
          dst += stage_bytes; fb += 8u; eb += 8u;
          if (++s == stages) { s = 0; ph ^= 1u; dst = base + box_off; fb = full_bar(0); eb = empty_bar(0); }
        }
      } else {
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u)) { ok = false; break; }
          if (lane == 0) mbar_expect_tx(full_bar(s), stage_bytes);
          int q[5];
#pragma unroll
          for (int d = 0; d < 5; ++d) q[d] = c[d] + (d == kd0 ? k0 : 0) + (d == kd1 ? k1 : 0);
          tma_load(base + uint32_t(s) * stage_bytes + box_off, map, full_bar(s), q[0], q[1], q[2], q[3], q[4]);
          k0 += BK; if (k0 >= x_k0) { k0 = 0; ++k1; }
          if (++s == stages) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x1u);
        *abort_flag = 1;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = make_idesc(bn, p.cfg.a_mn_major, p.cfg.b_mn_major);
      const uint32_t a_step = p.cfg.a_mn_major ? 128u : 2u, b_step = p.cfg.b_mn_major ? 128u : 2u;
      const uint64_t ad_first = make_desc(base, p.cfg.a_mn_major), bd_first = make_desc(base + kATileBytes, p.cfg.b_mn_major);
      const uint32_t a_hi = uint32_t(ad_first >> 32), b_hi = uint32_t(bd_first >> 32), stage16 = stage_bytes >> 4;
      uint32_t a_lo = uint32_t(ad_first), b_lo = uint32_t(bd_first);
      int s = 0;
      uint32_t ph = 0, accum = 0u;
      bool ok = true;
      for (int ks = 0; ks < ksteps; ++ks) {
        if (!mbar_wait(full_bar(s), ph)) { ok = false; break; }
        tc_fence_after();
        umma_bf16_lohi(tmem_base, a_lo, a_hi, b_lo, b_hi, idesc, accum);
        umma_bf16_lohi(tmem_base, a_lo + a_step, a_hi, b_lo + b_step, b_hi, idesc, 1u);
        umma_bf16_lohi(tmem_base, a_lo + 2u * a_step, a_hi, b_lo + 2u * b_step, b_hi, idesc, 1u);
        umma_bf16_lohi(tmem_base, a_lo + 3u * a_step, a_hi, b_lo + 3u * b_step, b_hi, idesc, 1u);
        umma_commit(empty_bar(s));
        accum = 1u;
        a_lo += stage16; b_lo += stage16;
        if (++s == stages) { s = 0; ph ^= 1u; a_lo = uint32_t(ad_first); b_lo = uint32_t(bd_first); }
      }
      if (ok) umma_commit(tfull);
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x2u);
        *abort_flag = 1;
      }
    }
  }
  const int rows_per = BM / sk;
  const uint32_t slice_bytes = uint32_t(rows_per) * uint32_t(bn) * 4u;
  bool have_acc = false;
  if (warp >= 2) {
    // ---------------- this CTA's partial tile -> shared memory, [128 rows][bn] fp32 over the drained stages ----------------
    have_acc = mbar_wait_warp(tfull, 0u);
    if (!have_acc && lane == 0) {
      if (!*abort_flag) atomicOr(p.status, 0x4u);
      *abort_flag = 1;
    }
    tc_fence_after();
    if (have_acc) {
      const int lane_base = (warp & 3) * 32, half = (warp - 2) >> 2;
      const int m_loc = lane_base + lane;                 // this thread's accumulator row
      const uint32_t row_addr = base + uint32_t(m_loc * bn) * 4u;
      const uint32_t trow = tmem_base + (uint32_t(lane_base) << 16);
      const int col_begin = half * (bn / 2), col_end = col_begin + bn / 2;
      uint32_t r[32];
      tmem_ld32(trow + uint32_t(col_begin), r);
#pragma unroll 1
      for (int c0 = col_begin; c0 < col_end; c0 += 32) {
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
        if (c0 + 32 < col_end) tmem_ld32(trow + uint32_t(c0 + 32), r);
#pragma unroll
        for (int u = 0; u < 8; ++u)   // 16-byte unit c4 of row m lives at unit c4 ^ (m & 7)
          sts128(row_addr + (uint32_t(((c0 >> 2) + u) ^ (m_loc & 7)) << 4), v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
      }
      tc_fence_before();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copies below read these writes
    }
  }
  __syncwarp();
  cluster_wait();   // every CTA of the cluster has started: its shared memory and barriers may be written
  // Second cluster barrier, arrival: "every slice sent to this CTA has landed", which is what the senders need to
  // know before their shared memory may go. Warps 0-1 have nothing to add and arrive now; the epilogue threads
  // arrive once the receive barrier has completed; everybody waits at the very end, after the stores.
  if (warp < 2) cluster_arrive();
  if (warp >= 2) {
    asm volatile("bar.sync 1, 256;" ::: "memory");   // the whole partial tile is in shared memory
    // rows [d * rows_per, ...) go to CTA d, into the slice that belongs to this CTA's rank; CTA r starts
    // with d = r and goes round, so that at any moment every CTA receives from one peer only
    if (warp == 2 && lane < sk && !*abort_flag) {
      const uint32_t d = uint32_t(sp + lane) & uint32_t(sk - 1);
      bulk_copy_to_cta(map_to_rank(recv + uint32_t(sp) * slice_bytes, d), base + d * slice_bytes, slice_bytes, map_to_rank(recv_bar, d));
    }
    // ---------------- reduce the split_k slices of this CTA's rows, epilogue, store ----------------
    const GemmParams& g = grp == 0 ? p.g : p.gx[grp - 1];
    const int t = threadIdx.x - 64;
    const int lg = bn == 64 ? 4 : 5;              // 16-byte units per row = bn / 4
    const int items = rows_per << lg;
    pdl_wait();  // before any global read (bias, residual) or write (C)
    const int64_t cbz = split_off(bz, g.B0, g.c_s[0], g.c_s[1]);
    const int64_t rbz = g.has_res ? split_off(bz, g.B0, g.r_s[0], g.r_s[1]) : 0;
    const int gM = g.M, gN = g.N, gM0 = g.M0;
    const int64_t cs2 = g.c_s[2], cs3 = g.c_s[3], rs2 = g.r_s[2], rs3 = g.r_s[3];
    const bool has_res = g.has_res != 0;
    FinalCtx f;
    f.C = g.C; f.R = g.R; f.bias = g.has_bias ? static_cast<const __nv_bfloat16*>(g.bias) : nullptr;
    f.cs4 = g.c_s[4]; f.rs4 = g.r_s[4]; f.N0 = g.N0; f.scale = g.scale;
    bool got = mbar_wait_warp(recv_bar, 0u);          // every peer's slice has landed (or a peer gave up)
    if (!got && lane == 0) {
      if (!*abort_flag) atomicOr(p.status, 0x8u);
      *abort_flag = 1;
    }
    cluster_arrive();
    if (got) {
      // two items per pass: their shared-memory reads and address arithmetic overlap
#pragma unroll 1
      for (int idx = t; idx < items; idx += 2 * kEpiWarps * 32) {
        float4 acc[2];
        int mm[2], nn[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int id = idx + j * kEpiWarps * 32;
          const int lr = id >> lg, c4 = id & ((1 << lg) - 1);
          mm[j] = id < items ? mt * BM + sp * rows_per + lr : gM;
          nn[j] = nt * bn + c4 * 4;
          const uint32_t a0 = recv + uint32_t(lr * bn) * 4u + (uint32_t(c4 ^ (lr & 7)) << 4);
          float4 part[8];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            part[q] = (q < sk && id < items) ? lds128_relaxed(a0 + uint32_t(q) * slice_bytes) : make_float4(0.f, 0.f, 0.f, 0.f);
          acc[j] = part[0];
#pragma unroll
          for (int q = 1; q < 8; ++q) { acc[j].x += part[q].x; acc[j].y += part[q].y; acc[j].z += part[q].z; acc[j].w += part[q].w; }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          if (mm[j] >= gM || nn[j] >= gN) continue;
          const int64_t cb = cbz + split_off(mm[j], gM0, cs2, cs3);
          const int64_t rb = has_res ? rbz + split_off(mm[j], gM0, rs2, rs3) : 0;
          final_store4_c<EPI>(f, acc[j], cb, rb, nn[j]);
        }
      }
    }
  }
  __syncwarp();
  cluster_wait();     // every peer has received what this CTA sent: its shared memory may go
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ---- CTA pair: two CTAs, one 256 x 256 output tile (tcgen05 cta_group::2) -------------------------------
// The single-CTA kernel pulls 48 KB from L2 per k-step of a 128 x 256 tile; with all SMs doing so the L2
// cannot keep the tensor cores fed. Here the two CTAs of a cluster share a 256 x 256 tile: each loads its
// own 128 rows of A and its own 128 columns of B (32 KB per k-step, six stages), and CTA 0 issues one
// 256 x 256 x 16 MMA that reads both CTAs' shared memory and writes rows 0-127 of the accumulator into its
// own tensor memory and rows 128-255 into its peer's. Barrier traffic across the pair:
//   full[s]    lives in CTA 0; the TMA loads of both CTAs complete on it (cta_group::2 loads)
//   empty[s]   in both CTAs; CTA 0's commit after a stage's MMAs arrives on both
//   tfull[a]   in both CTAs; CTA 0's commit after a tile's last MMA arrives on both
//   tempty[a]  lives in CTA 0; the epilogue warps of both CTAs arrive on it
// Every thread of both CTAs passes the cluster barriers at the start (barriers initialised) and at the end
// (tensor memory may be released) on every path; all mbarrier waits are bounded.
__device__ __forceinline__ void tma_load_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2,
                                              int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void umma_pair_bf16_lohi(uint32_t tmem_c, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                    uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n .reg .b64 da, db;\n mov.b64 da, {%1, %2};\n mov.b64 db, {%3, %4};\n setp.ne.b32 p, %6, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n}"
      ::"r"(tmem_c), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this shared-memory offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}

// SwiGLU epilogue of the CTA-pair kernel: accumulator columns [0, 128) hold the gate projection and [128, 256) the
// up projection of the same 128 output columns; the warp writes SiLU(gate) * up for its column range, through the
// same shared-memory turn as the other vector epilogues (bf16 output, n contiguous).
// Rotary embedding in the epilogue of a projection (rotate-half pairing, heads of 128 columns): a warp's half of a
// 256-wide tile is exactly one head, so columns d and d + 64 of a row sit in the same thread's accumulator row. Both
// 32-column chunks of a pair are read, rotated by the angle of the row's position (frequency table from the host,
// compensated fp32 angle product and reduction, as in the stand-alone kernel) and leave through the shared-memory turn of
// the other epilogues. The unrotated projection never exists in memory and is never rounded to bf16.
__device__ __forceinline__ void epilogue_tile_rope(const GemmParams& g, const RopeFreq& fr, uint32_t trow, int col_begin, int n_tile0,
                                                   const int64_t (&cbs)[8], uint32_t ok_mask, float* stage, int lane, int pos,
                                                   float row_scale = 1.f) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const float scale = g.scale * row_scale;
  __nv_bfloat16* const c_b16 = static_cast<__nv_bfloat16*>(g.C);
  if (n_tile0 + col_begin >= g.N) return;   // uniform across the warp
#pragma unroll 1
  for (int c0 = 0; c0 < 64; c0 += 32) {
    uint32_t ra[32], rb[32];
    tmem_ld32(trow + uint32_t(col_begin + c0), ra);
    tmem_ld32(trow + uint32_t(col_begin + 64 + c0), rb);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      float sn, cs;
      rope_sincos(pos, fr.hi[c0 + j], fr.lo[c0 + j], sn, cs);
      const float a = __uint_as_float(ra[j]) * scale, b = __uint_as_float(rb[j]) * scale;
      ra[j] = __float_as_uint(a * cs - b * sn);
      rb[j] = __float_as_uint(b * cs + a * sn);
    }
#pragma unroll
    for (int hsel = 0; hsel < 2; ++hsel) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t* r = hsel ? rb : ra;
        sts128(st_row + (uint32_t(u ^ (lane & 7)) << 4), __uint_as_float(r[4 * u]), __uint_as_float(r[4 * u + 1]),
               __uint_as_float(r[4 * u + 2]), __uint_as_float(r[4 * u + 3]));
      }
      __syncwarp();
      const int nc = n_tile0 + col_begin + hsel * 64 + c0 + unit * 4;
      int n1, n0i;
      split2(nc, g.N0, n1, n0i);
      const int64_t c_col = (int64_t)n1 * g.c_s[4] + n0i;
      const uint32_t live = nc < g.N ? ok_mask : 0u;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int row = rsub + 4 * i;
        const float4 v = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
        uint2* dst = reinterpret_cast<uint2*>(c_b16 + cbs[i] + c_col);
        const uint2 q = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
        if ((live >> i) & 1u) *dst = q;
      }
      __syncwarp();   // the staging tile is rewritten by the next turn
    }
  }
}

__device__ __forceinline__ void epilogue_tile_swiglu(const GemmParams& g, uint32_t trow, int col_begin, int col_end, int n_tile0,
                                                     const int64_t (&cbs)[8], uint32_t ok_mask, float* stage, int lane,
                                                     float row_scale = 1.f) {
  const int unit = lane & 7, rsub = lane >> 3;
  const uint32_t st_base = smem_u32(stage), st_row = st_base + uint32_t(lane) * 128u;
  const float scale = g.scale * row_scale;
  __nv_bfloat16* const c_b16 = static_cast<__nv_bfloat16*>(g.C);
#pragma unroll 1
  for (int c0 = col_begin; c0 < col_end; c0 += 32) {
    if (n_tile0 + c0 >= g.N) break;   // uniform across the warp
    uint32_t rg[32], ru[32];
    tmem_ld32(trow + uint32_t(c0), rg);
    tmem_ld32(trow + uint32_t(128 + c0), ru);
    tmem_ld_wait();
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      float o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) o[e] = silu(__uint_as_float(rg[4 * u + e]) * scale) * (__uint_as_float(ru[4 * u + e]) * scale);
      sts128(st_row + (uint32_t(u ^ (lane & 7)) << 4), o[0], o[1], o[2], o[3]);
    }
    __syncwarp();
    const int nc = n_tile0 + c0 + unit * 4;
    int n1, n0i;
    split2(nc, g.N0, n1, n0i);
    const int64_t c_col = (int64_t)n1 * g.c_s[4] + n0i;
    const uint32_t live = nc < g.N ? ok_mask : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = rsub + 4 * i;
      const float4 v = lds128(st_base + uint32_t(row * 128) + (uint32_t(unit ^ (row & 7)) << 4));
      uint2* dst = reinterpret_cast<uint2*>(c_b16 + cbs[i] + c_col);
      const uint2 q = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
      if ((live >> i) & 1u) *dst = q;
    }
    __syncwarp();   // the staging tile is rewritten by the next chunk
  }
}

template <int EPI>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                    const __grid_constant__ TcParams p) {
  // tile width of the pair (columns of the accumulator): 256, or 192 for plain steps whose tiles then fill one wave
  // (N = 768 over 16 row pairs: 64 tiles on 74 pairs instead of 48, each three quarters of the work)
  const int PN = (p.swiglu || EPI == EPI_ROPE) ? 256 : p.cfg.bn;
  constexpr uint32_t kBHalfBytes = 128 * BK * 2;   // room for this CTA's columns of the B tile (128 at most)
  constexpr uint32_t stage_bytes = kATileBytes + kBHalfBytes;
  const uint32_t stage_tx = kATileBytes + uint32_t(PN / 2) * BK * 2;   // bytes one CTA's loads of a stage bring
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const int stages = p.cfg.stages;
  const uint32_t bars = base + uint32_t(stages) * stage_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (stages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * stages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * stages + 2 + a); };
  const uint32_t tmem_slot = bars + 8u * (2 * stages + 4);
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  volatile uint32_t* abort_flag = tmem_slot_ptr + 1;
  const uint32_t stage_base = (tmem_slot + 16u + 15u) & ~15u;   // 8 warps x 4 KB epilogue staging tiles

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();            // 0: issues the MMAs; 1: its peer
  const int n_pairs = int(gridDim.x) >> 1, pair_id = int(blockIdx.x) >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
  }
  if (warp == 1) {   // the same warp of both CTAs: the allocation is made in both tensor memories at once
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();     // both CTAs' barriers are initialised before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  if (warp == 0) {
    // ---------------- TMA producer: one lane per box of this CTA's A rows / B columns ----------------
    const bool is_a = lane < 2;
    const int ch = is_a ? lane : lane - 2;
    const int box_rows = (is_a ? p.cfg.a_mn_major : p.cfg.b_mn_major) ? 64 : 128;
    const int n_box = 128 / box_rows;
    if (lane < 6 && ch < n_box) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      const uint32_t box_off = (is_a ? 0u : kATileBytes) + uint32_t(ch) * uint32_t(box_rows) * 128u;
      const int x_r0 = is_a ? p.cfg.a_r0 : p.cfg.b_r0, x_b0 = is_a ? p.cfg.a_b0 : p.cfg.b_b0;
      const int x_k0 = is_a ? p.cfg.a_k0 : p.cfg.b_k0;
      int sel[5];
#pragma unroll
      for (int d = 0; d < 5; ++d) sel[d] = is_a ? p.cfg.a_sel[d] : p.cfg.b_sel[d];
      int kd0 = 0, kd1 = -1;
#pragma unroll
      for (int d = 0; d < 5; ++d) {
        if (sel[d] == 0) kd0 = d;
        if (sel[d] == 1) kd1 = d;
      }
      const bool k_simple = kd1 < 0 && kd0 < 3;
      const int i0 = kd0 == 0 ? BK : 0, i1 = kd0 == 1 ? BK : 0, i2 = kd0 == 2 ? BK : 0;
      uint32_t dst = base + box_off, eb = empty_bar(0);
      uint32_t fb = map_to_rank(full_bar(0), 0u);       // the full barriers of CTA 0 collect both CTAs' bytes
      const uint32_t fb0 = fb;
      const bool b_free = p.g.b_const && (p.n_group < 2 || p.gx[0].b_const) && (p.n_group < 3 || p.gx[1].b_const);
      // A tile's coordinates are index arithmetic only (five divisions and the selects: ~1 us on this one warp), so the
      // first tile's are ready before the wait for the previous step and every later tile's while its predecessor's
      // loads are still in flight
      int c[5], ksteps = 0;
      const CUtensorMap* map = &map_a;
      auto prep = [&](int item) {
        int grp, bz, pm, nt;
        decode_tile(p, item, grp, bz, pm, nt);        // p.tiles_m counts pairs of row tiles here
        const int mt = 2 * pm + int(rank);
        ksteps = k_steps_of(p, mt);
        int r1, r0, b1, b0;
        split2((is_a ? mt * BM : (p.swiglu ? nt * 128 : nt * PN + int(rank) * (PN / 2))) + ch * box_rows, x_r0, r1, r0);
        split2(bz, x_b0, b1, b0);
        fill_coords(sel, 5, 0, 0, r0, r1, b0, b1, c);
        map = is_a ? &map_a : (p.swiglu ? (rank == 0 ? &map_b : &map_b1) : (grp == 0 ? &map_b : (grp == 1 ? &map_b1 : &map_b2)));
      };
      int item = pair_id;
      if (item < p.num_tiles) prep(item);
      if (is_a || !b_free) pdl_wait();   // weights do not wait for the previous step
      for (; ok && item < p.num_tiles; item += n_pairs, (item < p.num_tiles ? prep(item) : (void)0)) {
        int k0 = 0, k1 = 0;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(eb, ph ^ 1u)) { ok = false; break; }
          if (lane == 0 && rank == 0) mbar_expect_tx(full_bar(s), 2u * stage_tx);
          if (k_simple) {
            tma_load_pair(dst, map, fb, c[0], c[1], c[2], c[3], c[4]);
            c[0] += i0; c[1] += i1; c[2] += i2;
          } else {
            int q[5];
#pragma unroll
            for (int d = 0; d < 5; ++d) q[d] = c[d] + (d == kd0 ? k0 : 0) + (d == kd1 ? k1 : 0);
            tma_load_pair(dst, map, fb, q[0], q[1], q[2], q[3], q[4]);
            k0 += BK; if (k0 >= x_k0) { k0 = 0; ++k1; }
          }
          dst += stage_bytes; fb += 8u; eb += 8u;
          if (++s == stages) { s = 0; ph ^= 1u; dst = base + box_off; fb = fb0; eb = empty_bar(0); }
        }
      }
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x1u);
        *abort_flag = 1;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (CTA 0 only) ----------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(p.cfg.a_mn_major) << 15) |
                             (uint32_t(p.cfg.b_mn_major) << 16) | (uint32_t(PN >> 3) << 17) | (uint32_t(256 >> 4) << 24);
      const uint32_t a_step = p.cfg.a_mn_major ? 128u : 2u, b_step = p.cfg.b_mn_major ? 128u : 2u;
      const uint64_t ad_first = make_desc(base, p.cfg.a_mn_major), bd_first = make_desc(base + kATileBytes, p.cfg.b_mn_major);
      const uint32_t a_hi = uint32_t(ad_first >> 32), b_hi = uint32_t(bd_first >> 32);
      const uint32_t a_lo0 = uint32_t(ad_first), b_lo0 = uint32_t(bd_first), stage16 = stage_bytes >> 4;
      uint32_t a_lo = a_lo0, b_lo = b_lo0, fb = full_bar(0), eb = empty_bar(0);
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      bool ok = true;
      for (int item = pair_id; ok && item < p.num_tiles; item += n_pairs) {
        int grp, bz, pm, nt;
        decode_tile(p, item, grp, bz, pm, nt);
        const int ksteps = k_steps_of(p, 2 * pm);
        if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_c = tmem_base + uint32_t(acc * PN);
        uint32_t accum = 0u;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(fb, ph)) { ok = false; break; }
          tc_fence_after();
          umma_pair_bf16_lohi(tmem_c, a_lo, a_hi, b_lo, b_hi, idesc, accum);
          umma_pair_bf16_lohi(tmem_c, a_lo + a_step, a_hi, b_lo + b_step, b_hi, idesc, 1u);
          umma_pair_bf16_lohi(tmem_c, a_lo + 2u * a_step, a_hi, b_lo + 2u * b_step, b_hi, idesc, 1u);
          umma_pair_bf16_lohi(tmem_c, a_lo + 3u * a_step, a_hi, b_lo + 3u * b_step, b_hi, idesc, 1u);
          umma_commit_pair(eb);  // the stage is free in both CTAs once these MMAs have read it
          accum = 1u;
          a_lo += stage16; b_lo += stage16; fb += 8u; eb += 8u;
          if (++s == stages) { s = 0; ph ^= 1u; a_lo = a_lo0; b_lo = b_lo0; fb = full_bar(0); eb = empty_bar(0); }
        }
        if (ok) umma_commit_pair(tfull_bar(acc));  // accumulator complete, in both CTAs
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
      if (!ok) {
        if (!*abort_flag) atomicOr(p.status, 0x2u);
        *abort_flag = 1;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..9): this CTA's 128 rows of the tile ----------------
    const int lane_base = (warp & 3) * 32;
    const int half = (warp - 2) >> 2;
    float* stage = reinterpret_cast<float*>(smem_raw + (stage_base - raw)) + (warp - 2) * 1024;
    const int out_w = p.swiglu ? 128 : PN;   // output columns of a tile
    const int col_begin = half * (out_w / 2), col_end = col_begin + out_w / 2;
    int acc = 0;
    uint32_t acc_ph = 0;
    bool ok = true;
    bool waited = false;
    for (int item = pair_id; ok && item < p.num_tiles; item += n_pairs) {
      int grp, bz, pm, nt;
      decode_tile(p, item, grp, bz, pm, nt);
      const int mt = 2 * pm + int(rank);
      const GemmParams& g = grp == 0 ? p.g : p.gx[grp - 1];
      const int n_tile0 = nt * out_w;
      int64_t cbs[8], rbs[8];
      uint32_t ok_mask = 0;
      const int64_t cbz = split_off(bz, g.B0, g.c_s[0], g.c_s[1]);
      const int64_t rbz = g.has_res ? split_off(bz, g.B0, g.r_s[0], g.r_s[1]) : 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int mi = mt * BM + lane_base + (lane >> 3) + 4 * i;
        const bool live = mi < g.M;
        ok_mask |= live ? (1u << i) : 0u;
        cbs[i] = cbz + (live ? split_off(mi, g.M0, g.c_s[2], g.c_s[3]) : 0);
        rbs[i] = g.has_res ? rbz + (live ? split_off(mi, g.M0, g.r_s[2], g.r_s[3]) : 0) : 0;
      }
      // the first tile's row and column offsets above are index arithmetic (sixteen divisions): done before the wait
      if (!waited) { pdl_wait(); waited = true; }   // before any global read (bias, residual) or write (C)
      // second half of a split RMS normalisation: 1 / rms of this thread's accumulator row from the slabs its producer
      // left, in slab order (read while the tile's MMAs still run)
      float row_scale = 1.f;
      if ((EPI == EPI_SWIGLU || EPI == EPI_ROPE) && g.row_ss) {
        const int row = mt * BM + lane_base + lane;
        if (row < g.M) {
          const float* ssp = g.row_ss + (int64_t)row * g.row_slabs;
          float t = 0.f;
          for (int k = 0; k < g.row_slabs; k += 4) {
            const float4 q4 = *reinterpret_cast<const float4*>(ssp + k);
            t += q4.x; t += q4.y; t += q4.z; t += q4.w;
          }
          row_scale = rsqrtf(t * g.row_inv_n + g.row_eps);
        }
      }
      if (!mbar_wait_warp(tfull_bar(acc), acc_ph)) { ok = false; break; }
      tc_fence_after();
      const uint32_t trow = tmem_base + (uint32_t(lane_base) << 16) + uint32_t(acc * PN);
      if (EPI == EPI_SWIGLU) epilogue_tile_swiglu(g, trow, col_begin, col_end, n_tile0, cbs, ok_mask, stage, lane, row_scale);
      else if (EPI == EPI_ROPE) {
        if (g.rope) epilogue_tile_rope(g, p.rope_freq, trow, col_begin, n_tile0, cbs, ok_mask, stage, lane, (mt * BM + lane_base + lane) % g.rope_S, row_scale);
        else epilogue_tile_c<EPI_PLAIN>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, row_scale);
      } else if (EPI == EPI_RES_WIDE_NRM) epilogue_tile_resnorm(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane, mt * BM + lane_base);
      else epilogue_tile_c<EPI>(g, trow, col_begin, col_end, n_tile0, cbs, rbs, ok_mask, stage, lane);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(tempty_bar(acc), 0u));   // CTA 0 counts both CTAs' epilogue warps
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
    if (!ok && lane == 0) {
      if (!*abort_flag) atomicOr(p.status, 0x4u);
      *abort_flag = 1;
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();     // neither CTA releases tensor memory or leaves while its peer may still use it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace

bool tc_kernel_available() { return true; }

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

int encode_tensor_map(TensorMapStorage* out, const void* base, const TmaOperand& op) {
  static_assert(sizeof(CUtensorMap) == sizeof(TensorMapStorage), "tensor map size");
  EncodeTiledFn enc = get_encode();
  if (!enc || !base || (reinterpret_cast<uintptr_t>(base) & 15)) return -1;
  cuuint64_t dims[5], strides[4];
  cuuint32_t box[5], estr[5];
  for (int d = 0; d < 5; ++d) {  // unit dims pad every map to rank 5
    const bool real = d < op.rank;
    dims[d] = real ? op.dims[d] : 1;
    box[d] = real ? op.box[d] : 1;
    estr[d] = 1;
    if (d > 0) strides[d - 1] = (real ? op.strides[d] : 8) * 2;  // bytes
  }
  CUresult rc = enc(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : -2;
}

// A plain tiled map for copies: elements of `esize` bytes (2 or 4) moved as they are, dims / strides (bytes;
// strides[0] is ignored, the fastest dim is dense) / box given fastest first, padded to rank 5 by the caller.
// swizzle128: the 128-byte swizzle (box[0] * esize must then be 128 and the shared-memory box 1024-byte aligned).
int encode_tensor_map_plain(TensorMapStorage* out, const void* base, int esize, const uint64_t* dims, const uint64_t* strides_bytes,
                            const uint32_t* box, bool swizzle128) {
  EncodeTiledFn enc = get_encode();
  if (!enc || !base || (reinterpret_cast<uintptr_t>(base) & 15) || (esize != 2 && esize != 4)) return -1;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], estr[5];
  for (int i = 0; i < 5; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    estr[i] = 1;
    if (i > 0) st[i - 1] = strides_bytes[i];
  }
  CUresult rc = enc(reinterpret_cast<CUtensorMap*>(out), esize == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 5,
                    const_cast<void*>(base), d, st, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? 0 : -2;
}

// FLUID_PAIR=0 in the environment keeps every step on the single-CTA kernel.
static bool pair_enabled() {
  static int on = -1;
  if (on < 0) {
    const char* e = std::getenv("FLUID_PAIR");
    on = (e && e[0] == '0') ? 0 : 1;
  }
  return on == 1;
}

static bool vec_epilogue_ok(const GemmParams* gs, int n_group, bool check_pointers) {
  auto mult8 = [](int64_t v) { return (v & 7) == 0; };
  const GemmParams& g = gs[0];
  bool vec = true;
  for (int i = 0; i < n_group; ++i) {
    const GemmParams& q = gs[i];
    vec = vec && q.c_s[5] == 1 && (q.N & 7) == 0 && (q.N0 & 7) == 0 && mult8(q.c_s[0]) && mult8(q.c_s[1]) && mult8(q.c_s[2]) &&
          mult8(q.c_s[3]) && mult8(q.c_s[4]) && q.c_f32 == g.c_f32;
    if (check_pointers)
      vec = vec && (reinterpret_cast<uintptr_t>(q.C) & 15) == 0 && (!q.has_bias || (reinterpret_cast<uintptr_t>(q.bias) & 15) == 0);
  }
  if (g.has_res) {
    vec = vec && g.r_s[5] == 1 && mult8(g.r_s[0]) && mult8(g.r_s[1]) && mult8(g.r_s[2]) && mult8(g.r_s[3]) && mult8(g.r_s[4]);
    if (check_pointers) vec = vec && (reinterpret_cast<uintptr_t>(g.R) & 15) == 0;
    vec = vec && g.act == ACT_NONE && g.c_f32 == g.r_f32;
  } else if (g.act != ACT_NONE) {
    vec = vec && !g.c_f32;
  }
  return vec;
}

int gemm_split_k(const GemmParams& g, const GemmTcHost& tc, int n_group, int64_t* scratch_bytes) {
  *scratch_bytes = 0;
  if (g.causal != CAUSAL_NONE) return 1;
  GemmParams gs[3] = {g, g, g};
  if (!vec_epilogue_ok(gs, 1, false)) return 1;
  const int64_t tiles = int64_t((g.M + BM - 1) / BM) * ((g.N + tc.cfg.bn - 1) / tc.cfg.bn) * g.batch * n_group;
  const int ksteps = (g.K + BK - 1) / BK;
  if (tiles > 56 || tiles * 2 > sm_count() || ksteps < 16) return 1;
  int sk = (int)std::min<int64_t>(std::min<int64_t>(8, sm_count() / tiles), ksteps / 4);
  if (sk < 2) return 1;
  const int per = (ksteps + sk - 1) / sk;
  sk = (ksteps + per - 1) / per;   // no empty split
  if (sk < 2) return 1;
  *scratch_bytes = tiles * sk * int64_t(BM) * tc.cfg.bn * 4;
  return sk;
}

// Cluster size for the cluster split-K kernel, 0 if the step does not qualify: few output tiles (one
// wave of CTAs even after the split), at least two k-steps per CTA, no empty split, vector epilogue.
int gemm_cluster_split(const GemmParams* gs, const GemmTcHost& tc, int n_group) {
  const GemmParams& g = gs[0];
  if (g.causal != CAUSAL_NONE || tc.cfg.bn > 128 || tc.cfg.no_cluster) return 0;
  if (!vec_epilogue_ok(gs, n_group, false)) return 0;
  const int64_t tiles = int64_t((g.M + BM - 1) / BM) * ((g.N + tc.cfg.bn - 1) / tc.cfg.bn) * g.batch * n_group;
  const int ksteps = (g.K + BK - 1) / BK;
  // Clusters are placed whole inside a GPC (18-19 SMs of the 148), so a launch does not get all 148 SMs as clusters: launches
  // of 128 CTAs as sixteen clusters of 8 (N = 1024 in 64-wide tiles) and of 144 as thirty-six clusters of 4 measured as
  // if they ran in two waves (18.5 vs 13.5 us, 23.6 vs 15.1 us against the next narrower split); four fifths of the SMs fit.
  const int64_t cluster_sms = int64_t(sm_count()) * 4 / 5;
  for (int sk = 8; sk >= 2; sk >>= 1) {
    if (tiles * sk > cluster_sms || ksteps < 2 * sk) continue;
    const int per = (ksteps + sk - 1) / sk;
    if ((sk - 1) * per >= ksteps) continue;
    return sk;
  }
  return 0;
}

// True if the step runs as CTA pairs (two CTAs per 256 x 256 tile), decided from shapes and strides alone.
bool gemm_pair_eligible(const GemmParams* gs, const GemmTcHost& tc, int n_group) {
  const GemmParams& g = gs[0];
  if (!tc.cfg.pair || !pair_enabled() || g.causal != CAUSAL_NONE || ((g.M + BM - 1) / BM) % 2 != 0) return false;
  if (!vec_epilogue_ok(gs, n_group, false)) return false;
  return (g.act == ACT_NONE) || (!g.has_res && !g.c_f32);   // one of the templated epilogues applies
}

cudaError_t launch_gemm_tc(const GemmParams* gs, const GemmTcHost* tcs, int n_group, int split_k, int cluster_k, float* partial,
                           uint32_t* status, cudaStream_t stream, int swiglu, const RopeFreq* rope_freq) {
  const GemmParams& g = gs[0];
  const GemmTcHost& tc = tcs[0];
  TcParams p;
  p.g = g;
  p.n_group = n_group;
  for (int i = 1; i < 3; ++i) p.gx[i - 1] = gs[i < n_group ? i : 0];
  p.cfg = tc.cfg;
  p.tiles_m = (g.M + BM - 1) / BM;
  p.tiles_n = (g.N + tc.cfg.bn - 1) / tc.cfg.bn;
  long long per_batch = (long long)p.tiles_m * p.tiles_n;
  if (g.causal == CAUSAL_SKIP_UPPER) {
    per_batch = 0;
    for (int m = 0; m < p.tiles_m; ++m) per_batch += std::min(p.tiles_n, (m * BM + BM - 1) / tc.cfg.bn + 1);
  }
  if (per_batch * g.batch > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (per_batch * g.batch * n_group > 0x7fffffffLL) return cudaErrorInvalidValue;
  p.tiles_per_batch = (int)per_batch;
  p.tiles_per_group = (int)(per_batch * g.batch);
  p.num_tiles = p.tiles_per_group * n_group;
  p.status = status;
  p.swiglu = 0;
  const size_t smem = size_t(tc.cfg.stages) * (kATileBytes + size_t(tc.cfg.bn) * BK * 2) + 1024 + 8 * (2 * tc.cfg.stages + 4) + 16 +
                      16 + size_t(kEpiWarps) * 4096;
  const CUtensorMap* ma = reinterpret_cast<const CUtensorMap*>(&tc.map_a);
  const CUtensorMap* mb = reinterpret_cast<const CUtensorMap*>(&tc.map_b);
  const CUtensorMap* mb1 = reinterpret_cast<const CUtensorMap*>(&tcs[n_group > 1 ? 1 : 0].map_b);
  const CUtensorMap* mb2 = reinterpret_cast<const CUtensorMap*>(&tcs[n_group > 2 ? 2 : 0].map_b);
  // The vector epilogues need: n contiguous in C (and R), 8-column groups aligned to 16 bytes and
  // inside one n split, N a multiple of 8. Everything else takes the general epilogue.
  const bool vec = vec_epilogue_ok(gs, n_group, true);
  p.scalar_turn = 1;
  for (int i = 0; i < n_group; ++i)
    if (gs[i].c_s[5] != 1 || gs[i].N0 != gs[i].N || (gs[i].has_res && gs[i].r_s[5] != 1)) p.scalar_turn = 0;
  if (!vec || !partial) split_k = 1;   // the general epilogue does not take part in split-K
  p.split_k = split_k;
  p.partial = partial;
  {
    const int ksteps = (g.K + BK - 1) / BK;
    p.ksteps_per_split = (ksteps + split_k - 1) / split_k;
    if (split_k > 1) {
      if (p.num_tiles > 56) return cudaErrorInvalidValue;
      p.num_tiles *= split_k;
    }
  }
  int epi = EPI_ANY;
  if (vec) {
    if (g.act == ACT_NONE && !g.has_res) epi = g.c_f32 ? EPI_PLAIN_WIDE : EPI_PLAIN;
    else if (g.act == ACT_NONE && g.has_res && !g.c_f32 && !g.r_f32) epi = EPI_RES;
    else if (g.act == ACT_NONE && g.has_res && g.c_f32 && g.r_f32) epi = EPI_RES_WIDE;
    else if (g.act == ACT_GELU_ERF && !g.has_res && !g.c_f32) epi = EPI_GELU_ERF;
    else if (g.act == ACT_GELU_TANH && !g.has_res && !g.c_f32) epi = EPI_GELU_TANH;
  }
  // ---- few tiles: one cluster of CTAs per tile, split along k, reduced through distributed shared memory ----
  // (the caller chose cluster_k with gemm_cluster_split; it is re-derived here so that pointer alignment is checked too)
  const int csk = (cluster_k > 1 && vec && split_k <= 1 && epi != EPI_ANY) ? gemm_cluster_split(gs, tc, n_group) : 0;
  if (csk > 1 && p.num_tiles > 0) {
    p.split_k = csk;
    p.ksteps_per_split = ((g.K + BK - 1) / BK + csk - 1) / csk;
    p.cfg.stages = std::min(tc.cfg.bn == 64 ? 6 : 4, p.ksteps_per_split);
    const size_t csmem = size_t(p.cfg.stages) * (kATileBytes + size_t(tc.cfg.bn) * BK * 2) + size_t(BM) * tc.cfg.bn * 4 + 1024 +
                         8 * (2 * p.cfg.stages + 1) + 16;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(p.num_tiles * csk));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = csmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = unsigned(csk); attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    static bool cattr_set[7] = {false, false, false, false, false, false, false};
#define FLUID_TC_CLUSTER(E)                                                                                          \
  case E: {                                                                                                          \
    if (!cattr_set[E]) {                                                                                             \
      cudaError_t e = cudaFuncSetAttribute(gemm_tc_cluster_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024); \
      if (e != cudaSuccess) return e;                                                                                \
      cattr_set[E] = true;                                                                                           \
    }                                                                                                                \
    return cudaLaunchKernelEx(&cfg, gemm_tc_cluster_kernel<E>, *ma, *mb, *mb1, *mb2, p);                             \
  }
    switch (epi) {
      FLUID_TC_CLUSTER(EPI_PLAIN)
      FLUID_TC_CLUSTER(EPI_PLAIN_WIDE)
      FLUID_TC_CLUSTER(EPI_RES)
      FLUID_TC_CLUSTER(EPI_RES_WIDE)
      FLUID_TC_CLUSTER(EPI_GELU_ERF)
      FLUID_TC_CLUSTER(EPI_GELU_TANH)
      default: break;
    }
#undef FLUID_TC_CLUSTER
  }
  // ---- many 256-wide tiles over an even number of row tiles: pairs of CTAs share 256 x 256 tiles ----
  if (swiglu && !(tc.cfg.pair && pair_enabled() && vec && n_group == 2 && (p.tiles_m & 1) == 0)) return cudaErrorInvalidValue;
  bool rope = false;
  for (int i = 0; i < n_group; ++i) rope = rope || gs[i].rope;
  if (rope) {   // the rotary epilogue exists in the CTA-pair form only, over the plain bf16 epilogue
    if (!(tc.cfg.pair && pair_enabled() && vec && epi == EPI_PLAIN && !swiglu && rope_freq && (p.tiles_m & 1) == 0 &&
          g.causal == CAUSAL_NONE && split_k <= 1))
      return cudaErrorInvalidValue;
    for (int i = 0; i < n_group; ++i)
      if (gs[i].rope && (gs[i].N0 % 128 != 0 || gs[i].N % 128 != 0 || gs[i].rope_S < 1 || gs[i].batch != 1)) return cudaErrorInvalidValue;
    p.rope_freq = *rope_freq;
    epi = EPI_ROPE;
  }
  if (tc.cfg.pair && pair_enabled() && vec && epi != EPI_ANY && split_k <= 1 && g.causal == CAUSAL_NONE && (p.tiles_m & 1) == 0 &&
      p.num_tiles > 0) {
    TcParams q = p;
    q.tiles_m = p.tiles_m / 2;                       // pairs of row tiles
    if (swiglu) {                                    // one tile = 128 output columns = 128 gate + 128 up accumulator columns
      q.swiglu = 1;
      q.tiles_n = (g.N + 127) / 128;
      epi = EPI_SWIGLU;
    }
    q.tiles_per_batch = q.tiles_m * q.tiles_n;
    q.tiles_per_group = q.tiles_per_batch * g.batch;
    q.num_tiles = q.tiles_per_group * (swiglu ? 1 : n_group);
    q.cfg.stages = 6;
    q.split_k = 1;
    const size_t psmem = size_t(q.cfg.stages) * (kATileBytes + size_t(128) * BK * 2) + 1024 + 8 * (2 * q.cfg.stages + 4) + 16 + 16 +
                         size_t(kEpiWarps) * 4096;
    const int n_pairs = std::min(q.num_tiles, sm_count() / 2);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(2 * n_pairs));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = psmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    static bool pattr_set[10] = {};
#define FLUID_TC_PAIR(E)                                                                                             \
  case E: {                                                                                                          \
    if (!pattr_set[E]) {                                                                                             \
      cudaError_t e = cudaFuncSetAttribute(gemm_tc_pair_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024); \
      if (e != cudaSuccess) return e;                                                                                \
      pattr_set[E] = true;                                                                                           \
    }                                                                                                                \
    return cudaLaunchKernelEx(&cfg, gemm_tc_pair_kernel<E>, *ma, *mb, *mb1, *mb2, q);                                \
  }
    if (g.nrm_out) {   // first half of a split RMS normalisation: whole 256-wide tiles of one fp32 residual stream
      if (epi != EPI_RES_WIDE || n_group != 1 || !g.nrm_gamma || !g.nrm_ss || g.N % 256 != 0 || g.N0 != g.N || tc.cfg.bn != 256)
        return cudaErrorInvalidValue;
      epi = EPI_RES_WIDE_NRM;
    }
    switch (epi) {
      FLUID_TC_PAIR(EPI_PLAIN)
      FLUID_TC_PAIR(EPI_PLAIN_WIDE)
      FLUID_TC_PAIR(EPI_RES)
      FLUID_TC_PAIR(EPI_RES_WIDE)
      FLUID_TC_PAIR(EPI_RES_WIDE_NRM)
      FLUID_TC_PAIR(EPI_GELU_ERF)
      FLUID_TC_PAIR(EPI_GELU_TANH)
      FLUID_TC_PAIR(EPI_SWIGLU)
      FLUID_TC_PAIR(EPI_ROPE)
      default: break;
    }
#undef FLUID_TC_PAIR
  }
  if (tc.cfg.bn == 192) return cudaErrorInvalidValue;   // the 192-wide tile exists in the CTA-pair form only
  for (int i = 0; i < n_group; ++i)
    if (gs[i].nrm_out || gs[i].row_ss) return cudaErrorInvalidValue;   // so does the split normalisation
  const int grid = std::min(p.num_tiles, sm_count());
  if (grid <= 0) return cudaSuccess;
  static bool attr_set[7] = {false, false, false, false, false, false, false};
#define FLUID_TC_LAUNCH(E)                                                                                           \
  case E: {                                                                                                          \
    if (!attr_set[E]) {                                                                                              \
      cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<E, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024); \
      if (e == cudaSuccess)                                                                                          \
        e = cudaFuncSetAttribute(gemm_tc_kernel<E, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);  \
      if (e != cudaSuccess) return e;                                                                                \
      attr_set[E] = true;                                                                                            \
    }                                                                                                                \
    return split_k > 1 ? launch_k(gemm_tc_kernel<E, true>, grid, kThreads, smem, stream, *ma, *mb, *mb1, *mb2, p)    \
                       : launch_k(gemm_tc_kernel<E, false>, grid, kThreads, smem, stream, *ma, *mb, *mb1, *mb2, p);                                   \
  }
  switch (epi) {
    FLUID_TC_LAUNCH(EPI_PLAIN)
    FLUID_TC_LAUNCH(EPI_PLAIN_WIDE)
    FLUID_TC_LAUNCH(EPI_RES)
    FLUID_TC_LAUNCH(EPI_RES_WIDE)
    FLUID_TC_LAUNCH(EPI_GELU_ERF)
    FLUID_TC_LAUNCH(EPI_GELU_TANH)
    default:
      FLUID_TC_LAUNCH(EPI_ANY)
  }
#undef FLUID_TC_LAUNCH
  return cudaSuccess;
}

}  // namespace fluid

// ---- a GEMM entry point that allocates nothing -----------------------------------------------------
// The split-K kernel needs scratch for its partial tiles and arrival counters. Inside a plan that
// scratch is a slice of the caller's arena. A caller with no arena and no licence to allocate (see
// fluid.h) gets it from this fixed array, which every GPU that loads the library keeps until exit.
namespace fluid {
namespace {
constexpr size_t kStaticHeaderBytes = 256;                 // status word + arrival counters
constexpr size_t kStaticPartialBytes = size_t(8) << 20;    // 8 MiB of fp32 partial tiles
static __device__ __align__(256) unsigned char g_static_scratch[kStaticHeaderBytes + kStaticPartialBytes];
// g_static_scratch is only a host-side handle here; the device address is looked up once per device.
std::mutex g_static_mu;
void* g_static_addr[64] = {};
}  // namespace
}  // namespace fluid

extern "C" int fluid_gemm_bf16_static_scratch(const void* dev_a, const void* dev_b, const void* dev_bias, void* dev_c,
                                              int m, int n, int k, fluid_stream stream) {
  using namespace fluid;
  if (!dev_a || !dev_b || !dev_c || m < 1 || n < 1 || k < 1) {
    set_error("static-scratch GEMM: null operand or empty shape");
    return FLUID_EINVAL;
  }
  if ((k & 7) || (n & 7)) {
    set_error("static-scratch GEMM: K and N must be multiples of 8 (got K=%d, N=%d)", k, n);
    return FLUID_EINVAL;
  }
  const uintptr_t align_bits = reinterpret_cast<uintptr_t>(dev_a) | reinterpret_cast<uintptr_t>(dev_b) |
                               reinterpret_cast<uintptr_t>(dev_c) | reinterpret_cast<uintptr_t>(dev_bias);
  if (align_bits & 15) {
    set_error("static-scratch GEMM: device pointers must be 16-byte aligned");
    return FLUID_EALIGN;
  }
  GemmParams g{};
  g.A = dev_a; g.B = dev_b; g.C = dev_c; g.bias = dev_bias;
  g.dtype = FLUID_BF16;
  g.M = m; g.N = n; g.K = k; g.batch = 1;
  g.M0 = m; g.N0 = n; g.K0 = k; g.B0 = 1;
  g.a_s[3] = k; g.a_s[5] = 1;   // A[m, k], k contiguous
  g.b_s[3] = 1; g.b_s[5] = k;   // B[n, k], k contiguous
  g.c_s[3] = n; g.c_s[5] = 1;   // C[m, n], n contiguous
  g.scale = 1.f;
  g.has_bias = dev_bias != nullptr;
  GemmTcHost tc;
  if (!gemm_tc_describe(g, &tc)) {
    set_error("static-scratch GEMM: shape %dx%dx%d cannot be fed to the tensor-core kernel", m, n, k);
    return FLUID_EUNSUPPORTED;
  }
  int64_t need = 0;
  const int split_k = gemm_split_k(g, tc, 1, &need);
  if ((size_t)need > kStaticPartialBytes) {
    set_error("static-scratch GEMM: %dx%dx%d needs %lld bytes of split-K scratch, the static array holds %zu", m, n, k,
              (long long)need, kStaticPartialBytes);
    return FLUID_EINVAL;
  }
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess || dev < 0 || dev >= 64) {
    set_error("static-scratch GEMM: no current device (%s)", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  unsigned char* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_addr[dev]) {   // first call on this device: resolve the array's device address
      void* ptr = nullptr;
      err = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (err != cudaSuccess || !ptr) {
        set_error("static-scratch GEMM: cudaGetSymbolAddress failed (%s)", cudaGetErrorString(err));
        return FLUID_ECUDA;
      }
      g_static_addr[dev] = ptr;
    }
    scratch = static_cast<unsigned char*>(g_static_addr[dev]);
  }
  if (encode_tensor_map(&tc.map_a, dev_a, tc.a) != 0 || encode_tensor_map(&tc.map_b, dev_b, tc.b) != 0) {
    set_error("static-scratch GEMM: tensor map encoding failed");
    return FLUID_ECUDA;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the last call left: status word and arrival counters must start at zero
  err = cudaMemsetAsync(scratch, 0, kStaticHeaderBytes, st);
  if (err == cudaSuccess)
    err = launch_gemm_tc(&g, &tc, 1, split_k, 0, reinterpret_cast<float*>(scratch + kStaticHeaderBytes),
                         reinterpret_cast<uint32_t*>(scratch), st);
  if (err != cudaSuccess) {
    set_error("static-scratch GEMM: %s", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  return FLUID_OK;
}

extern "C" int fluid_static_scratch_status(fluid_stream stream, int* device_status) {
  using namespace fluid;
  if (!device_status) {
    set_error("static-scratch status: null argument");
    return FLUID_EINVAL;
  }
  *device_status = 0;
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess || dev < 0 || dev >= 64) {
    set_error("static-scratch status: no current device (%s)", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  void* addr = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_static_mu);
    addr = g_static_addr[dev];
  }
  err = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  uint32_t word = 0;
  // no call on this device yet: the array was never handed to a kernel, nothing to read
  if (err == cudaSuccess && addr) err = cudaMemcpy(&word, addr, sizeof(word), cudaMemcpyDeviceToHost);
  if (err != cudaSuccess) {
    set_error("static-scratch status: %s", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  *device_status = (int)word;
  if (word != 0) {
    set_error("static-scratch GEMM: a device-side wait expired (code 0x%x); the output is incomplete", word);
    return FLUID_ETIMEOUT;
  }
  return FLUID_OK;
}
