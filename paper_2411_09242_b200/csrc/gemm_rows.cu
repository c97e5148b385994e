// GEMM with a handful of rows (M <= 16: the LINEAR steps of single-token decoding). The step reads every
// weight once and does M multiply-adds per weight, so it is bound by streaming the weight matrix from HBM,
// not by arithmetic: a 128-row tcgen05 tile would stage 16x more rows than exist through shared memory and
// tensor memory and pay that pipeline's fill and drain per short k range. Here every warp streams 16 weight rows
// through a ring of its own in shared memory and feeds them to the arithmetic as they land. Two forms of the ring:
// bulk-tensor boxes of 16 rows x 64 k brought in by the TMA unit (gemm_rows_tma_kernel, the one that runs), and
// 16-byte asynchronous copies, every lane fetching what it will consume itself (gemm_rows_kernel: weights whose
// n index is not one flat stride, rows too long for the boxes' ring beside the staged activations, or
// FLUID_ROWS_TMA=0).
//
// C[m, n] = epilogue(scale * sum_k X[m, k] * W[n, k]), X = the step's A operand (k contiguous), W = its B operand
// held k-contiguous ("column-major" in the paper's matmul figure).
//
// The multiply-adds use the warp-level m16n8k16 bf16 MMA with fp32 accumulation as the arithmetic unit, with the
// roles swapped: 16 weight rows are the MMA's row operand, the activation rows its 8 columns (two MMAs side by side
// for 9 to 16 activation rows). The
// contraction index may be fed in any order as long as both operands agree, so a lane takes 8 *consecutive* k of
// one weight row (one 16-byte copy) and the same 8 k of one activation row, and two MMAs consume them: no
// unpacking, no shuffles, no exchange between lanes.
//
// A warp owns 16 weight rows and a slice of the k range; the warps that share a tile add their partial sums
// through shared memory and the CTA's threads apply bias / activation / residual and store.
// Sibling projections that share X (Q/K/V, gate/up) run as one launch (blockIdx.y = group).
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

constexpr int kWarps = 16;         // one CTA per SM: 16 warps, each streaming its own weight rows
constexpr int kBlk = 32;           // k per pass: 4 lanes x 8 elements per weight row
constexpr int kXPad = 32;          // bf16 elements of padding per staged activation row (64 bytes: rows g and g + 1 then sit 16
                                   // banks apart, so the eight lanes of a 16-byte shared load never collide)
constexpr int kSmemBudget = 227 * 1024 - 1024;

struct RowsGroup {
  const __nv_bfloat16* W;
  void* C;
  const __nv_bfloat16* bias;
  const void* R;
  int64_t b_s4, b_s5;      // weight row strides of the two-level n index
  int64_t c_s[6], r_s[6];
  int c_f32, r_f32, has_bias, has_res, act;
};

struct RowsParams {
  const void* X;           // bf16, or fp32 when x_f32
  int M, N, K, M0, N0;
  int64_t a_s2, a_s3;      // activation row strides of the two-level m index
  const __nv_bfloat16* gamma;   // fused normalisation: the gain (else null)
  const __nv_bfloat16* beta;    // fused LayerNorm: the bias (null: RMS normalisation)
  float eps;
  int x_f32;
  float scale;
  int w_const;             // the weights are constants of the plan: their first loads need not wait
  int tiles, units, upc, rounds;   // 16-row weight tiles per group; (group, tile) units in all; units per CTA and round; rounds
  RowsGroup g[3];
};

__device__ __forceinline__ int64_t split2(int i, int x0, int64_t s1, int64_t s0) {
  if (i < x0) return (int64_t)i * s0;
  const int hi = i / x0;
  return (int64_t)hi * s1 + (int64_t)(i - hi * x0) * s0;
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool ok) {
  const int bytes = ok ? 16 : 0;   // 0: the 16 bytes are zero-filled, nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");   // past L1: read once
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

// Stages the step's activation rows in shared memory as bf16, once per CTA (all threads of the CTA call this; it
// ends before the block-wide barrier that must precede the first read of xs / rstd). pitch = bf16 elements between
// staged rows; the pad_chunks 8-element pieces after a row's K elements are zeroed (they meet zero weights when the
// last pass of k reaches past K). part: 16 floats of scratch; rstd: the rows' 1 / rms (1 without a normalisation).
__device__ __forceinline__ void stage_activations(const RowsParams& p, __nv_bfloat16* xs, int pitch, int pad_chunks, float* part,
                                                  float* rstd) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ln = p.beta ? 1 : 0;
  // ---- stage the activations: thread -> 8 consecutive k of one row ----
  // The 16 warps are dealt to the rows (the LayerNorm bias counts as one): 16 / rows warps each, rounded down to a
  // power of two; a row's statistics go through a few words of shared memory.
  // LayerNorm: ((x - mean) * rstd * gamma + beta) . W = rstd * (((x - mean) * gamma) . W) + beta . W. The rows are
  // centred and multiplied by the gain here; the bias rides along as one more activation row (an MMA column that
  // would otherwise be idle), so beta . W comes out of the same accumulators.
  const int chunks = p.K / 8;
  const int n_rows = p.M + ln;
  const int wpr = n_rows > 8 ? 1 : (n_rows > 4 ? 2 : (n_rows > 2 ? 4 : (n_rows > 1 ? 8 : 16)));
  const int row = warp / wpr, c0 = (warp % wpr) * 32 + lane, cstep = 32 * wpr;
  const bool is_x = row < p.M, is_beta = ln && row == p.M;
  auto load_x8 = [&](int64_t off, float (&xf)[8]) {
    if (p.x_f32) {
      const float4 lo = *reinterpret_cast<const float4*>(static_cast<const float*>(p.X) + off);
      const float4 hi = *reinterpret_cast<const float4*>(static_cast<const float*>(p.X) + off + 4);
      xf[0] = lo.x; xf[1] = lo.y; xf[2] = lo.z; xf[3] = lo.w; xf[4] = hi.x; xf[5] = hi.y; xf[6] = hi.z; xf[7] = hi.w;
    } else {
      load16(static_cast<const __nv_bfloat16*>(p.X) + off, xf);
    }
  };
  const int64_t roff = is_x ? split2(row, p.M0, p.a_s2, p.a_s3) : 0;
  __nv_bfloat16* dst = xs + size_t(row < n_rows ? row : 0) * pitch;
  float mean = 0.f;
  if (ln) {
    float sm = 0.f;
    if (is_x) {
#pragma unroll 4
      for (int c = c0; c < chunks; c += cstep) {
        float xf[8];
        load_x8(roff + c * 8, xf);
#pragma unroll
        for (int i = 0; i < 8; ++i) sm += xf[i];
      }
    }
    sm = warp_sum(sm);
    if (lane == 0) part[warp] = sm;
    __syncthreads();
    if (is_x) {
      float tot = 0.f;
      for (int q = 0; q < wpr; ++q) tot += part[row * wpr + q];
      mean = tot / p.K;
    }
    __syncthreads();   // the words are reused for the sums of squares
  }
  float acc = 0.f;
  if (is_x) {
#pragma unroll 4
    for (int c = c0; c < chunks; c += cstep) {
      uint4 out;
      if (p.gamma || p.x_f32) {
        float xf[8];
        load_x8(roff + c * 8, xf);
        if (p.gamma) {
          float gf[8];
          load16(p.gamma + c * 8, gf);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            xf[i] -= mean;
            acc = fmaf(xf[i], xf[i], acc);
            xf[i] *= gf[i];
          }
        }
        out = make_uint4(pack_bf16x2(xf[0], xf[1]), pack_bf16x2(xf[2], xf[3]), pack_bf16x2(xf[4], xf[5]), pack_bf16x2(xf[6], xf[7]));
      } else {
        out = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.X) + roff + c * 8);
      }
      *reinterpret_cast<uint4*>(dst + c * 8) = out;
    }
  } else if (is_beta) {
    for (int c = c0; c < chunks; c += cstep) *reinterpret_cast<uint4*>(dst + c * 8) = *reinterpret_cast<const uint4*>(p.beta + c * 8);
  }
  // the padding is read (against zero weights) when K is not a multiple of 32
  if ((is_x || is_beta) && warp % wpr == 0 && lane < pad_chunks) *reinterpret_cast<uint4*>(dst + (chunks + lane) * 8) = make_uint4(0u, 0u, 0u, 0u);
  acc = warp_sum(acc);
  if (lane == 0) part[warp] = acc;
  __syncthreads();
  if (threadIdx.x < p.M) {
    float q2 = 0.f;
    for (int q = 0; q < wpr; ++q) q2 += part[threadIdx.x * wpr + q];
    rstd[threadIdx.x] = p.gamma ? rsqrtf(q2 / p.K + p.eps) : 1.f;
  }
}

// One CTA per SM. The CTA first stages the activation rows in shared memory, once, as bf16 (with the RMS
// normalisation's gain multiplied in and the rows' 1/rms computed when the step carries the normalisation): every
// warp of the GPU reading the same few rows from L2 pass by pass was measured to cost more L2 traffic than the
// weights themselves and to serialise on the lines everybody wants at once. Then every warp takes work items
// (16-row weight tile, k slice): KS warps share a tile, the weights of a slice go through a per-lane ring in shared
// memory filled by 16-byte asynchronous copies (a lane only ever reads back what it copied itself, so the ring needs
// no barrier; the bytes in flight are set by the ring's depth, not by registers), the activation fragment comes from
// the staged copy. ST = ring depth. SWIGLU: groups 0 and 1 are the gate and up projections; the same tiles of both
// sit in neighbouring warps and the CTA writes SiLU(gate) * up to group 0's C, so neither projection is ever stored.
// MT = 8-row groups of activation rows (1: M <= 8, 2: M <= 16; a second MMA column block).
template <int KS, int ST, bool SWIGLU, int MT>
__global__ void __launch_bounds__(kWarps * 32, 1) gemm_rows_kernel(RowsParams p) {
  constexpr int MC = 8 * MT;                       // activation rows the accumulators cover
  constexpr int NG = SWIGLU ? 2 : 1;               // groups inside a CTA
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = p.K + kXPad;                   // staged activation row, bf16 elements
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  const int ln = p.beta ? 1 : 0;                   // LayerNorm: one more staged row (the bias), see below
  unsigned char* after_x = smem_raw + size_t(p.M + ln) * pitch * 2;
  const uint32_t ring0 = static_cast<uint32_t>(__cvta_generic_to_shared(after_x));
  // partial sums [row][m] of a warp: laid over the warp's own ring, which is drained by the time they are written
  auto red = [&](int w) { return reinterpret_cast<float(*)[MC + 1]>(after_x + size_t(w) * (ST * 1024)); };
  float* rstd = reinterpret_cast<float*>(after_x + kWarps * ST * 1024);   // [16]
  float* part = rstd + 16;                                                // [16]: per-warp sums while staging
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int nblk = (p.K + kBlk - 1) / kBlk;
  const int per = (nblk + KS - 1) / KS;
  const int ks = warp % KS;
  const int blk0 = ks * per;
  const uint32_t my_ring = ring0 + uint32_t(warp) * (ST * 1024) + uint32_t(lane) * 16;
  auto slot = [&](int i, int piece) { return my_ring + uint32_t(i % ST) * 1024 + uint32_t(piece) * 512; };
  const uint32_t xs_lane = static_cast<uint32_t>(__cvta_generic_to_shared(xs)) + uint32_t((g < p.M + ln ? g : 0) * pitch + t * 8) * 2;
  const bool x_live = g < p.M + ln;
  const bool x_live2 = MT == 2 && g + 8 < p.M + ln;   // activation rows 8 .. 15

  for (int round = 0; round < p.rounds; ++round) {
    // units are dealt out evenly: a CTA takes p.upc <= UMAX of them per round, so that every SM streams
    const int ul = warp / (KS * NG);
    const int unit = (round * p.upc + ul) * gridDim.x + blockIdx.x;   // strided: CTA c takes units c, c + grid, ...
    const bool live = ul < p.upc && unit < p.units;
    const int tile = SWIGLU ? unit : unit % p.tiles;
    const RowsGroup& grp = p.g[SWIGLU ? (warp / KS) % 2 : (live ? unit / p.tiles : 0)];
    const int blk1 = live ? min(nblk, blk0 + per) : blk0;
    const int nloc = max(0, blk1 - blk0);
    const int n_base = tile * 16;
    // weight rows of this lane: g and g + 8 of the tile (rows past N read row N-1 and are dropped at the end)
    const __nv_bfloat16* wrow[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int n = max(0, min(p.N - 1, n_base + hh * 8 + g));
      wrow[hh] = grp.W + split2(n, p.N0, grp.b_s4, grp.b_s5) + t * 8;
    }
    auto fill_w = [&](int i) {
      const int k = (blk0 + i) * kBlk;
      const bool ok = i < nloc && k + t * 8 < p.K;   // K is a multiple of 8: a piece is all inside or all outside
      const int kk = ok ? k : 0;
      cp_async16(slot(i, 0), wrow[0] + kk, ok);
      cp_async16(slot(i, 1), wrow[1] + kk, ok);
    };
    // constant weights do not depend on the previous step: the ring fills while the activations are staged
    if (round > 0 || p.w_const) {
      for (int i = 0; i < ST - 1; ++i) {
        fill_w(i);
        cp_async_commit();
      }
    }
    if (round == 0) {
      pdl_wait();
      if (!p.w_const) {
        for (int i = 0; i < ST - 1; ++i) {
          fill_w(i);
          cp_async_commit();
        }
      }
      stage_activations(p, xs, pitch, kXPad / 8, part, rstd);
      // (rstd is read after the __syncthreads that follows the main loop)
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int i = 0; i < nloc; ++i) {
      cp_async_wait<ST - 2>();   // this lane's copies of pass i have landed
      const uint4 w0 = lds128(slot(i, 0)), w1 = lds128(slot(i, 1));
      const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
      const uint4 x = x_live ? lds128(xs_lane + uint32_t(blk0 + i) * (kBlk * 2)) : zero4;
      uint4 x2 = zero4;
      if (MT == 2 && x_live2) x2 = lds128(xs_lane + uint32_t(8 * pitch * 2) + uint32_t(blk0 + i) * (kBlk * 2));
      fill_w(i + ST - 1);        // refills the slot read one pass ago
      cp_async_commit();
      mma_bf16(acc, w0.x, w1.x, w0.y, w1.y, x.x, x.y);
      mma_bf16(acc, w0.z, w1.z, w0.w, w1.w, x.z, x.w);
      if (MT == 2) {
        mma_bf16(acc2, w0.x, w1.x, w0.y, w1.y, x2.x, x2.y);
        mma_bf16(acc2, w0.z, w1.z, w0.w, w1.w, x2.z, x2.w);
      }
    }
    cp_async_wait<0>();
    // accumulator fragment: acc[0..1] = (weight row g; activation rows 2t, 2t+1), acc[2..3] = (weight row g + 8; same)
    red(warp)[g][2 * t] = acc[0];
    red(warp)[g][2 * t + 1] = acc[1];
    red(warp)[g + 8][2 * t] = acc[2];
    red(warp)[g + 8][2 * t + 1] = acc[3];
    if (MT == 2) {
      red(warp)[g][8 + 2 * t] = acc2[0];
      red(warp)[g][8 + 2 * t + 1] = acc2[1];
      red(warp)[g + 8][8 + 2 * t] = acc2[2];
      red(warp)[g + 8][8 + 2 * t + 1] = acc2[3];
    }
    __syncthreads();
    // thread -> (tile of the CTA, m, row of the tile) with the row fastest, so that stores to an n-contiguous C coalesce
    for (int e = threadIdx.x; e < p.upc * 16 * MC; e += kWarps * 32) {
      const int nl = e % 16, m = (e / 16) % MC, tl = e / (16 * MC);
      const int u = (round * p.upc + tl) * gridDim.x + blockIdx.x;
      if (u >= p.units) continue;
      const int n = (SWIGLU ? u : u % p.tiles) * 16 + nl;
      if (m >= p.M || n >= p.N) continue;
      const float sc = p.scale * rstd[m];
      float v = 0.f;
#pragma unroll
      for (int q = 0; q < KS; ++q) v += red(tl * NG * KS + q)[nl][m];
      v *= sc;
      if (SWIGLU) {
        float u = 0.f;
#pragma unroll
        for (int q = 0; q < KS; ++q) u += red((tl * NG + 1) * KS + q)[nl][m];
        v = silu(v) * (u * sc);
      }
      if (ln) {   // + beta . W
        float bw = 0.f;
#pragma unroll
        for (int q = 0; q < KS; ++q) bw += red(tl * NG * KS + q)[nl][p.M];
        v = fmaf(bw, p.scale, v);
      }
      const RowsGroup& og = p.g[SWIGLU ? 0 : u / p.tiles];
      if (og.has_bias) v += __bfloat162float(og.bias[n]);
      if (og.act == ACT_GELU_ERF) v = gelu_erf(v);
      else if (og.act == ACT_GELU_TANH) v = gelu_tanh(v);
      if (og.has_res) {
        const int64_t ro = split2(m, p.M0, og.r_s[2], og.r_s[3]) + split2(n, p.N0, og.r_s[4], og.r_s[5]);
        v += og.r_f32 ? static_cast<const float*>(og.R)[ro] : __bfloat162float(static_cast<const __nv_bfloat16*>(og.R)[ro]);
      }
      const int64_t co = split2(m, p.M0, og.c_s[2], og.c_s[3]) + split2(n, p.N0, og.c_s[4], og.c_s[5]);
      if (og.c_f32) static_cast<float*>(og.C)[co] = v;
      else static_cast<__nv_bfloat16*>(og.C)[co] = __float2bfloat16_rn(v);
    }
    __syncthreads();   // the partial sums are overwritten by the next round
  }
}

// ---- the same step with the weights brought in by the TMA unit ----
// What bounds the streaming is the order in which HBM is swept: a kernel that only pulls the Llama head (262 MB) through
// shared memory in this kernel's tile pattern reaches 5.4 TB/s when every warp walks the whole k range of its own
// 16 rows and 6.0 TB/s when the 16 warps of a CTA split the k range of ONE tile, i.e. the CTA reads 16 x K
// contiguous elements at a time (a plain coalesced sweep of the same bytes: 6.3). So here KS is as large as K
// allows (up to all 16 warps on a tile), a CTA walks its tiles round after round, and a warp's ring keeps
// running across the rounds: while the CTA adds up and stores the partial sums of one round, the first boxes of
// the next are already in flight.
//
// A box is 16 weight rows x 64 k (2 KB, 128-byte rows, 128-byte swizzle); a stage is nb of them side by side along
// k; lane 0 of a warp issues the loads of a stage and re-arms its barrier, all lanes wait on the barrier and read
// their fragments. In pass sb (0, 1) of a box lane (g, t) takes the 16-byte chunk 2t + sb of rows g and g + 8:
// the swizzle puts chunk c of row r at (c ^ (r & 7)), so the eight lanes of a quarter warp (g = 2q, 2q + 1;
// t = 0..3) hit eight different bank groups; the activation rows are staged with a pitch of 16 bytes mod 128 for
// the same reason. As in the kernel above, the contraction index is fed in an order both operands share.
constexpr int kBoxK = 64;                 // k per box
constexpr uint32_t kBoxBytes = 16 * kBoxK * 2;
constexpr int kMaxStages = 4;
constexpr long long kWaitCycles = 3000000000LL;

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

struct RowsTma {
  int nb, stages, ks;      // boxes per stage; stages in a warp's ring; warps that share a tile
  int pitch;               // staged activation row, bf16 elements
  uint32_t* status;        // bit 0x800: a bounded wait expired
};

template <bool SWIGLU, int MT>
__global__ void __launch_bounds__(kWarps * 32, 1)
gemm_rows_tma_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
                     const __grid_constant__ CUtensorMap map2, const __grid_constant__ RowsParams p,
                     const __grid_constant__ RowsTma q) {
  constexpr int MC = 8 * MT;
  constexpr int NG = SWIGLU ? 2 : 1;
  extern __shared__ __align__(1024) unsigned char smem_boxes[];
  const uint32_t raw = static_cast<uint32_t>(__cvta_generic_to_shared(smem_boxes));
  const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;       // boxes must sit on 1024-byte boundaries
  unsigned char* base = smem_boxes + pad;
  const int ln = p.beta ? 1 : 0;
  const uint32_t stage_bytes = kBoxBytes * uint32_t(q.nb);
  const uint32_t ring_bytes = uint32_t(kWarps * q.stages) * stage_bytes;
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(base + ring_bytes);                       // [16][kMaxStages]
  // partial sums [warp][row][m], two copies that take turns: a round's sums are read while the next round's are written
  constexpr uint32_t kRedBytes = uint32_t(kWarps) * 16 * (MC + 1) * 4;
  int rb = 0;
  auto red = [&](int w) {
    return reinterpret_cast<float(*)[MC + 1]>(base + ring_bytes + kWarps * kMaxStages * 8 + uint32_t(rb) * kRedBytes) + size_t(w) * 16;
  };
  float* rstd = reinterpret_cast<float*>(base + ring_bytes + kWarps * kMaxStages * 8 + 2 * kRedBytes);   // [16]
  float* part = rstd + 16;                                                                                                     // [16]
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(part + 16);
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const uint32_t ring = raw + pad + uint32_t(warp * q.stages) * stage_bytes;
  const uint32_t bars = static_cast<uint32_t>(__cvta_generic_to_shared(bar_mem)) + uint32_t(warp * kMaxStages) * 8u;
  if (lane == 0) {
    for (int s = 0; s < q.stages; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8u * s), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 3) {
    const CUtensorMap* m = threadIdx.x == 0 ? &map0 : (threadIdx.x == 1 ? &map1 : &map2);
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
  }
  __syncwarp();

  // this warp's share: k stages [k0, k0 + nk) of the tiles of units (r upc + ul) grid + cta, r = 0, 1, ...
  const int stage_k = kBoxK * q.nb;
  const int nk_all = (p.K + stage_k - 1) / stage_k;
  const int per = (nk_all + q.ks - 1) / q.ks;
  const int ksl = warp % q.ks;
  const int k0 = ksl * per;
  const int nk = max(0, min(nk_all, k0 + per) - k0);
  const int ul = warp / (q.ks * NG);
  const int gsel = SWIGLU ? (warp / q.ks) % 2 : 0;
  auto unit_of = [&](int r) { return (r * p.upc + ul) * int(gridDim.x) + int(blockIdx.x); };
  int my_rounds = 0;
  if (ul < p.upc)
    while (my_rounds < p.rounds && unit_of(my_rounds) < p.units) ++my_rounds;
  const int total = my_rounds * nk;
  // the next stage to request: lane 0 walks (round, k stage) by increments
  int is_r = 0, is_j = 0, issued = 0;
  auto issue = [&]() {
    const int u = unit_of(is_r);
    const int tile = SWIGLU ? u : u % p.tiles;
    const int grp = SWIGLU ? gsel : u / p.tiles;
    const CUtensorMap* m = grp == 0 ? &map0 : (grp == 1 ? &map1 : &map2);
    const int s = issued % q.stages;
    const uint32_t bar = bars + 8u * s, dst = ring + uint32_t(s) * stage_bytes;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(stage_bytes) : "memory");
    for (int b = 0; b < q.nb; ++b)
      asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %5, %5}], [%2];"
                   ::"r"(dst + uint32_t(b) * kBoxBytes), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"((k0 + is_j) * stage_k + b * kBoxK),
                     "r"(tile * 16), "r"(0) : "memory");
    ++issued;
    if (++is_j == nk) { is_j = 0; ++is_r; }
  };
  // constant weights do not depend on the previous step: the ring fills while the activations are staged
  if (p.w_const && lane == 0)
    while (issued < q.stages && issued < total) issue();
  pdl_wait();
  if (!p.w_const && lane == 0)
    while (issued < q.stages && issued < total) issue();
  stage_activations(p, xs, q.pitch, (q.pitch - p.K) / 8, part, rstd);
  __syncthreads();

  const uint32_t xs_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(xs));
  const bool x_live = g < p.M + ln;
  const bool x_live2 = MT == 2 && g + 8 < p.M + ln;
  const uint32_t xs_lane = xs_u32 + uint32_t((x_live ? g : 0) * q.pitch) * 2u + uint32_t(t) * 32u;
  const uint32_t w_lane = uint32_t(g) * 128u;
  const uint32_t sw0 = uint32_t((2 * t) ^ g) << 4, sw1 = uint32_t((2 * t + 1) ^ g) << 4;
  bool ok = true;
  int done = 0;   // stages consumed
  for (int round = 0; round < p.rounds; ++round) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc2[4] = {0.f, 0.f, 0.f, 0.f};
    if (ok && round < my_rounds) {
#pragma unroll 1
      for (int j = 0; j < nk; ++j, ++done) {
        const int s = done % q.stages;
        // one answer per warp: the lanes meet again at the __syncwarp below
        ok = __all_sync(0xffffffffu, mbar_wait(bars + 8u * s, uint32_t(done / q.stages) & 1u));
        if (!ok) break;
        const uint32_t wst = ring + uint32_t(s) * stage_bytes + w_lane;
        const uint32_t xst = xs_lane + uint32_t((k0 + j) * stage_k) * 2u;
        for (int b = 0; b < q.nb; ++b) {
#pragma unroll
          for (int sb = 0; sb < 2; ++sb) {
            const uint32_t wa = wst + uint32_t(b) * kBoxBytes + (sb ? sw1 : sw0);
            const uint4 w0 = lds128(wa), w1 = lds128(wa + 1024u);
            const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
            const uint32_t xa = xst + uint32_t(b) * (kBoxK * 2) + uint32_t(sb) * 16u;
            const uint4 x = x_live ? lds128(xa) : zero4;
            mma_bf16(acc, w0.x, w1.x, w0.y, w1.y, x.x, x.y);
            mma_bf16(acc, w0.z, w1.z, w0.w, w1.w, x.z, x.w);
            if (MT == 2) {
              const uint4 x2 = x_live2 ? lds128(xa + uint32_t(8 * q.pitch) * 2u) : zero4;
              mma_bf16(acc2, w0.x, w1.x, w0.y, w1.y, x2.x, x2.y);
              mma_bf16(acc2, w0.z, w1.z, w0.w, w1.w, x2.z, x2.w);
            }
          }
        }
        __syncwarp();   // every lane has read the stage: it may be refilled
        if (lane == 0 && issued < total) issue();
      }
    }
    // accumulator fragment: acc[0..1] = (weight row g; activation rows 2t, 2t+1), acc[2..3] = (weight row g + 8; same)
    red(warp)[g][2 * t] = acc[0];
    red(warp)[g][2 * t + 1] = acc[1];
    red(warp)[g + 8][2 * t] = acc[2];
    red(warp)[g + 8][2 * t + 1] = acc[3];
    if (MT == 2) {
      red(warp)[g][8 + 2 * t] = acc2[0];
      red(warp)[g][8 + 2 * t + 1] = acc2[1];
      red(warp)[g + 8][8 + 2 * t] = acc2[2];
      red(warp)[g + 8][8 + 2 * t + 1] = acc2[3];
    }
    __syncthreads();
    // thread -> (tile of the CTA, m, row of the tile) with the row fastest, so that stores to an n-contiguous C coalesce
    for (int e = threadIdx.x; e < p.upc * 16 * MC; e += kWarps * 32) {
      const int nl = e % 16, m = (e / 16) % MC, tl = e / (16 * MC);
      const int u = (round * p.upc + tl) * int(gridDim.x) + int(blockIdx.x);
      if (u >= p.units) continue;
      const int n = (SWIGLU ? u : u % p.tiles) * 16 + nl;
      if (m >= p.M || n >= p.N) continue;
      const float sc = p.scale * rstd[m];
      float v = 0.f;
      for (int k = 0; k < q.ks; ++k) v += red(tl * NG * q.ks + k)[nl][m];
      v *= sc;
      if (SWIGLU) {
        float up = 0.f;
        for (int k = 0; k < q.ks; ++k) up += red((tl * NG + 1) * q.ks + k)[nl][m];
        v = silu(v) * (up * sc);
      }
      if (ln) {   // + beta . W
        float bw = 0.f;
        for (int k = 0; k < q.ks; ++k) bw += red(tl * NG * q.ks + k)[nl][p.M];
        v = fmaf(bw, p.scale, v);
      }
      const RowsGroup& og = p.g[SWIGLU ? 0 : u / p.tiles];
      if (og.has_bias) v += __bfloat162float(og.bias[n]);
      if (og.act == ACT_GELU_ERF) v = gelu_erf(v);
      else if (og.act == ACT_GELU_TANH) v = gelu_tanh(v);
      if (og.has_res) {
        const int64_t ro = split2(m, p.M0, og.r_s[2], og.r_s[3]) + split2(n, p.N0, og.r_s[4], og.r_s[5]);
        v += og.r_f32 ? static_cast<const float*>(og.R)[ro] : __bfloat162float(static_cast<const __nv_bfloat16*>(og.R)[ro]);
      }
      const int64_t co = split2(m, p.M0, og.c_s[2], og.c_s[3]) + split2(n, p.N0, og.c_s[4], og.c_s[5]);
      if (og.c_f32) static_cast<float*>(og.C)[co] = v;
      else static_cast<__nv_bfloat16*>(og.C)[co] = __float2bfloat16_rn(v);
    }
    rb ^= 1;   // (this copy is written again two rounds on, past the next round's barrier)
  }
  if (!ok) {
    // a wait ran out: report it, and let the loads still in flight land (bounded again) before the shared memory is given up
    if (lane == 0) {
      if (q.status) atomicOr(q.status, 0x800u);
      for (; done < issued; ++done) mbar_wait(bars + 8u * (done % q.stages), uint32_t(done / q.stages) & 1u);
    }
  }
}

// staged rows (the LayerNorm bias counts as a row) + 1/rms and the staging sums (the partial sums of the epilogue lie
// over the rings)
inline size_t rows_fixed_smem(int rows, int K) { return size_t(rows) * (K + kXPad) * 2 + 32 * sizeof(float); }
constexpr int kRingMin = 5;   // fewest ring stages worth running with

template <int KS, int ST, bool SWIGLU, int MT>
cudaError_t launch_rows_mt(RowsParams& p, int n_group, cudaStream_t st) {
  const size_t smem = rows_fixed_smem(p.M + (p.beta ? 1 : 0), p.K) + size_t(kWarps) * ST * 1024;
  static const cudaError_t attr =
      cudaFuncSetAttribute(gemm_rows_kernel<KS, ST, SWIGLU, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
  if (attr != cudaSuccess) return attr;
  constexpr int UMAX = kWarps / (KS * (SWIGLU ? 2 : 1));
  p.units = SWIGLU ? p.tiles : p.tiles * n_group;
  const int grid = std::min(148, p.units);
  p.upc = std::min(UMAX, (p.units + grid - 1) / grid);
  p.rounds = (p.units + grid * p.upc - 1) / (grid * p.upc);
  return launch_k(gemm_rows_kernel<KS, ST, SWIGLU, MT>, dim3((unsigned)grid), dim3(kWarps * 32), smem, st, p);
}

template <int KS, int ST, bool SWIGLU>
cudaError_t launch_rows(RowsParams& p, int n_group, cudaStream_t st) {
  return p.M + (p.beta ? 1 : 0) > 8 ? launch_rows_mt<KS, ST, SWIGLU, 2>(p, n_group, st) : launch_rows_mt<KS, ST, SWIGLU, 1>(p, n_group, st);
}

template <int ST>
cudaError_t launch_rows_ks(RowsParams& p, int n_group, bool swiglu, cudaStream_t st) {
  // as many warps per tile (k slices) as keep the whole launch in one round of the grid
  const int64_t items = (int64_t)p.tiles * n_group, cap = 148 * kWarps;
  if (swiglu) {
    if (items * 8 <= cap) return launch_rows<8, ST, true>(p, n_group, st);
    if (items * 4 <= cap) return launch_rows<4, ST, true>(p, n_group, st);
    if (items * 2 <= cap) return launch_rows<2, ST, true>(p, n_group, st);
    return launch_rows<1, ST, true>(p, n_group, st);
  }
  if (items * 16 <= cap) return launch_rows<16, ST, false>(p, n_group, st);
  if (items * 8 <= cap) return launch_rows<8, ST, false>(p, n_group, st);
  if (items * 4 <= cap) return launch_rows<4, ST, false>(p, n_group, st);
  if (items * 2 <= cap) return launch_rows<2, ST, false>(p, n_group, st);
  return launch_rows<1, ST, false>(p, n_group, st);
}

inline bool flat(int X, int X0, int64_t s1, int64_t s0) { return X0 >= X || s1 == (int64_t)X0 * s0; }
inline bool al16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

// Which form runs. By default the TMA form takes the launches that stream at least kTmaMinBytes of weights: there the
// order of the sweep decides (kernel durations, cold caches: 4 x 32000 x 4096, 262 MB, 46.3 us against 53.5 us by
// per-lane copies; 4 x 22016 x 4096, 180 MB, 35.4 against 37.5), while a short stream is bound by how soon its first
// bytes arrive, and the per-lane form starts sooner (4 x 4096 x 4096, 34 MB: 11.0 us against 13.4; 4 x 50257 x 768,
// 77 MB: 21.5 against 26.2). FLUID_ROWS_TMA=0: never; =1: whenever the step qualifies; ="nb,stages,ks": ditto, with
// that geometry (boxes per stage, stages per warp, warps per tile).
constexpr int64_t kTmaMinBytes = int64_t(128) << 20;
struct RowsTmaEnv { bool on, always; int nb, stages, ks; };
inline RowsTmaEnv rows_tma_env() {
  RowsTmaEnv e{true, false, 0, 0, 0};
  if (const char* s = std::getenv("FLUID_ROWS_TMA")) {
    int a = -1, b = 0, c = 0;
    const int n = std::sscanf(s, "%d,%d,%d", &a, &b, &c);
    if (n == 1 && a == 0) e.on = false;
    if (n == 1 && a == 1) e.always = true;
    if (n == 3) { e.always = true; e.nb = a; e.stages = b; e.ks = c; }
  }
  return e;
}

inline size_t rows_tma_smem(int rows, int pitch, int nb, int stages, int mc) {
  return 1024 + size_t(kWarps) * stages * nb * kBoxBytes + kWarps * kMaxStages * 8 + 2 * size_t(kWarps) * 16 * (mc + 1) * 4 + 32 * sizeof(float) +
         size_t(rows) * pitch * 2;
}

template <bool SWIGLU, int MT>
cudaError_t launch_tma_k(int grid, size_t smem, cudaStream_t st, const CUtensorMap* m, const RowsParams& p, const RowsTma& q) {
  static const cudaError_t attr =
      cudaFuncSetAttribute(gemm_rows_tma_kernel<SWIGLU, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
  if (attr != cudaSuccess) return attr;
  return launch_k(gemm_rows_tma_kernel<SWIGLU, MT>, dim3((unsigned)grid), dim3(kWarps * 32), smem, st, m[0], m[1], m[2], p, q);
}

// The TMA form: false if the step does not qualify (nothing launched; the caller runs the per-lane form).
bool launch_rows_tma(RowsParams& p, int n_group, bool swiglu, uint32_t* status, cudaStream_t st, cudaError_t* err) {
  const RowsTmaEnv env = rows_tma_env();
  if (!env.on) return false;
  if (!env.always && int64_t(n_group) * p.N * p.K * 2 < kTmaMinBytes) return false;
  const int rows = p.M + (p.beta ? 1 : 0), mt = rows > 8 ? 2 : 1, ng = swiglu ? 2 : 1;
  // every group's weight: one flat n index with 16-byte aligned rows
  TensorMapStorage maps[3];
  for (int i = 0; i < n_group; ++i) {
    const RowsGroup& g = p.g[i];
    if (!flat(p.N, p.N0, g.b_s4, g.b_s5)) return false;
    const uint64_t row_b = p.N > 1 ? uint64_t(g.b_s5) * 2 : uint64_t(p.K) * 2;
    if ((row_b & 15) || row_b >= (uint64_t(1) << 40) || row_b < uint64_t(p.K) * 2) return false;
    uint64_t dims[5] = {(uint64_t)p.K, (uint64_t)p.N, 1, 1, 1}, str[5] = {2, row_b, row_b, row_b, row_b};
    uint32_t box[5] = {(uint32_t)kBoxK, 16, 1, 1, 1};
    if (encode_tensor_map_plain(&maps[i], g.W, 2, dims, str, box, true) != 0) return false;
  }
  for (int i = n_group; i < 3; ++i) maps[i] = maps[0];
  RowsTma q{};
  q.status = status;
  // boxes per stage: two (a 256-byte run of every row) unless K is short; warps per tile: up to 8, as many as leave
  // each at least two stages of k
  q.nb = env.nb > 0 ? env.nb : (p.K >= 2048 ? 2 : 1);
  const int stage_k = kBoxK * q.nb, nk_all = (p.K + stage_k - 1) / stage_k;
  q.ks = 1;
  while (q.ks * 2 <= 8 && q.ks * 2 * 2 <= nk_all) q.ks *= 2;   // (16 warps on a tile measured no faster than 8)
  if (env.ks > 0) q.ks = env.ks;
  if (q.ks < 1 || q.ks > kWarps / ng || (q.ks & (q.ks - 1)) || q.nb < 1 || q.nb > 4) return false;
  q.pitch = nk_all * stage_k + 8;    // 16 bytes mod 128: see the kernel
  // ring: 128 KB a CTA when it fits beside the staged rows (deeper rings measured no faster), 64 KB at least
  q.stages = env.stages > 0 ? env.stages : std::max(2, 4 / q.nb);
  if (q.stages > kMaxStages) q.stages = kMaxStages;
  while (q.stages > 2 && rows_tma_smem(rows, q.pitch, q.nb, q.stages, 8 * mt) > size_t(kSmemBudget)) --q.stages;
  if (rows_tma_smem(rows, q.pitch, q.nb, q.stages, 8 * mt) > size_t(kSmemBudget)) {
    if (env.nb > 0 || q.nb == 1) return false;
    q.nb = 1;     // (pitch and ks stay valid: the k range is cut into twice as many stages)
    q.stages = 3;
    while (q.stages > 2 && rows_tma_smem(rows, q.pitch, q.nb, q.stages, 8 * mt) > size_t(kSmemBudget)) --q.stages;
    if (rows_tma_smem(rows, q.pitch, q.nb, q.stages, 8 * mt) > size_t(kSmemBudget)) return false;
  }
  const size_t smem = rows_tma_smem(rows, q.pitch, q.nb, q.stages, 8 * mt);
  const int umax = kWarps / (q.ks * ng);
  p.units = swiglu ? p.tiles : p.tiles * n_group;
  const int grid = std::min(148, p.units);
  p.upc = std::min(umax, (p.units + grid - 1) / grid);
  p.rounds = (p.units + grid * p.upc - 1) / (grid * p.upc);
  const CUtensorMap* m = reinterpret_cast<const CUtensorMap*>(maps);
  static_assert(sizeof(TensorMapStorage) == sizeof(CUtensorMap), "tensor map storage");
  if (swiglu) *err = mt == 2 ? launch_tma_k<true, 2>(grid, smem, st, m, p, q) : launch_tma_k<true, 1>(grid, smem, st, m, p, q);
  else *err = mt == 2 ? launch_tma_k<false, 2>(grid, smem, st, m, p, q) : launch_tma_k<false, 1>(grid, smem, st, m, p, q);
  return true;
}

}  // namespace

bool gemm_rows_eligible(const GemmParams& g) {
  if (g.dtype != FLUID_BF16 || g.batch != 1 || g.M < 1 || g.M > 16 || g.causal != CAUSAL_NONE) return false;
  if (g.K % 8 || g.K < 8) return false;
  // the activation rows are staged in shared memory next to a ring of at least five stages per warp
  // (with more than 8 rows the tcgen05 path is no slower than this kernel on a five-stage ring: ask for seven)
  if (rows_fixed_smem(g.M, g.K) + size_t(kWarps) * (g.M > 8 ? 7 : kRingMin) * 1024 > size_t(kSmemBudget)) return false;
  // both operands with a flat, contiguous k index
  if (g.a_s[5] != 1 || !flat(g.K, g.K0, g.a_s[4], 1)) return false;
  if (g.b_s[3] != 1 || !flat(g.K, g.K0, g.b_s[2], 1)) return false;
  // 16-byte loads: every row starts on a 16-byte boundary
  const int64_t rows[4] = {g.M > g.M0 ? g.a_s[2] : 0, g.M > 1 ? g.a_s[3] : 0, g.N > g.N0 ? g.b_s[4] : 0, g.N > 1 ? g.b_s[5] : 0};
  for (int64_t s : rows)
    if (s % 8) return false;
  return true;
}

cudaError_t launch_gemm_rows(const GemmParams* gs, int n_group, cudaStream_t st, int swiglu, const RowsNorm* norm, uint32_t* status) {
  if (n_group < 1 || n_group > 3 || (swiglu && n_group != 2)) return cudaErrorInvalidValue;
  const GemmParams& g0 = gs[0];
  RowsParams p{};
  p.X = norm ? norm->x : g0.A;
  p.x_f32 = norm ? norm->x_f32 : 0;
  p.gamma = norm ? static_cast<const __nv_bfloat16*>(norm->gamma) : nullptr;
  p.beta = norm ? static_cast<const __nv_bfloat16*>(norm->beta) : nullptr;
  if (p.beta && (swiglu || g0.M > 15 || !al16(p.beta))) return cudaErrorInvalidValue;
  p.eps = norm ? norm->eps : 0.f;
  p.M = g0.M; p.N = g0.N; p.K = g0.K; p.M0 = g0.M0; p.N0 = g0.N0;
  p.a_s2 = g0.a_s[2]; p.a_s3 = g0.a_s[3];
  p.scale = g0.scale;
  p.w_const = 1;
  if (!al16(p.X) || (norm && !al16(norm->gamma))) return cudaErrorInvalidValue;
  for (int i = 0; i < n_group; ++i) {
    const GemmParams& g = gs[i];
    if (!gemm_rows_eligible(g) || g.M != g0.M || g.N != g0.N || g.K != g0.K || g.N0 != g0.N0 || g.M0 != g0.M0 || !al16(g.B))
      return cudaErrorInvalidValue;
    RowsGroup& q = p.g[i];
    q.W = static_cast<const __nv_bfloat16*>(g.B);
    q.C = g.C;
    q.bias = static_cast<const __nv_bfloat16*>(g.bias);
    q.R = g.R;
    q.b_s4 = g.b_s[4]; q.b_s5 = g.b_s[5];
    for (int j = 0; j < 6; ++j) { q.c_s[j] = g.c_s[j]; q.r_s[j] = g.r_s[j]; }
    q.c_f32 = g.c_f32; q.r_f32 = g.r_f32; q.has_bias = g.has_bias; q.has_res = g.has_res; q.act = g.act;
    p.w_const = p.w_const && g.b_const;
  }
  p.tiles = (p.N + 15) / 16;
  {
    cudaError_t err = cudaSuccess;
    if (launch_rows_tma(p, n_group, swiglu != 0, status, st, &err)) return err;
  }
  // ring depth: what the staged activations leave (one 16-byte piece per lane, row and stage; wider pieces measured
  // three times slower: a copy instruction of the warp then touches every 32-byte sector half)
  const size_t fixed = rows_fixed_smem(p.M + (p.beta ? 1 : 0), p.K);
  if (fixed + size_t(kWarps) * kRingMin * 1024 > size_t(kSmemBudget)) return cudaErrorInvalidValue;
  const size_t left = size_t(kSmemBudget) - fixed;
  if (left >= size_t(kWarps) * 10 * 1024) return launch_rows_ks<10>(p, n_group, swiglu != 0, st);
  if (left >= size_t(kWarps) * 7 * 1024) return launch_rows_ks<7>(p, n_group, swiglu != 0, st);
  return launch_rows_ks<kRingMin>(p, n_group, swiglu != 0, st);
}

}  // namespace fluid
