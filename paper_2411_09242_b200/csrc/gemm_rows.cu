// GEMM with a handful of rows (M <= 8: the LINEAR steps of single-token decoding). The step reads every
// weight once and does M multiply-adds per weight, so it is bound by streaming the weight matrix from HBM,
// not by arithmetic: a 128-row tcgen05 tile would stage 16x more rows than exist through shared memory and
// tensor memory and pay that pipeline's fill and drain per short k range. Here every lane copies the 16 bytes it
// will consume itself (asynchronous copies into a private ring in shared memory, five deep) and feeds them to the
// arithmetic as they land.
//
// C[m, n] = epilogue(scale * sum_k X[m, k] * W[n, k]), X = the step's A operand (k contiguous), W = its B operand
// held k-contiguous ("column-major" in the paper's matmul figure).
//
// The multiply-adds use the warp-level m16n8k16 bf16 MMA with fp32 accumulation as the arithmetic unit, with the
// roles swapped: 16 weight rows are the MMA's row operand, the (up to 8) activation rows its 8 columns. The
// contraction index may be fed in any order as long as both operands agree, so a lane takes 8 *consecutive* k of
// one weight row (one 16-byte copy) and the same 8 k of one activation row, and two MMAs consume them: no
// unpacking, no shuffles, no exchange between lanes.
//
// A warp owns 16 weight rows and a slice of the k range; the warps that share a tile add their partial sums
// through shared memory and the CTA's threads apply bias / activation / residual and store.
// Sibling projections that share X (Q/K/V, gate/up) run as one launch (blockIdx.y = group).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

// warps of a CTA: the KS warps of one tile (times two with SwiGLU: gate and up), at least two. Small CTAs spread the
// tiles evenly over the SMs: with eight-warp CTAs a launch of 250 CTAs left a third of the SMs with half the work.
__host__ __device__ constexpr int rows_warps(int ks, bool swiglu) { return ks * (swiglu ? 2 : 1) < 2 ? 2 : ks * (swiglu ? 2 : 1); }
constexpr int kWarpsPerSm = 24;   // resident warps an SM's shared memory holds rings for

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
  const __nv_bfloat16* X;
  int M, N, K, M0, N0;
  int64_t a_s2, a_s3;      // activation row strides of the two-level m index
  float scale;
  int w_const;             // the weights are constants of the plan: their first loads need not wait
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

// A warp's work item is (16-row weight tile, k slice): KS warps share a tile, a CTA holds 8 / KS tiles. The weights
// of a slice go through a per-lane ring in shared memory filled by 16-byte asynchronous copies (a lane only ever
// reads back what it copied itself, so the ring needs no barrier): the bytes in flight are set by the ring's
// depth, not by registers.

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

// LW = 16-byte pieces a lane takes of each row per stage (a stage covers 32 * LW k: 4 lanes x 8 * LW contiguous
// elements per row), ST = ring depth.
// SWIGLU: groups 0 and 1 are the gate and up projections; a CTA holds the same tiles of both (their warps side by
// side) and writes SiLU(gate) * up to group 0's C, so neither projection is ever stored.
template <int KS, int LW, int ST, bool SWIGLU>
__global__ void __launch_bounds__(rows_warps(KS, SWIGLU) * 32) gemm_rows_kernel(RowsParams p, int tiles) {
  constexpr int kWarps = rows_warps(KS, SWIGLU);
  constexpr int kBlk = 32 * LW, kStages = ST;
  constexpr int kStageBytes = 3 * LW * 32 * 16;
  constexpr int NG = SWIGLU ? 2 : 1;               // groups inside a CTA
  constexpr int TPC = kWarps / (KS * NG);          // tiles per CTA
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // ring: [warp][stage][3 = weight row g, weight row g + 8, activation row g][lane] x 16 bytes
  const uint32_t ring0 = static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw));
  float(*red)[16][9] = reinterpret_cast<float(*)[16][9]>(smem_raw + kWarps * kStages * kStageBytes);   // [warp][row][m]
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int tile = blockIdx.x * TPC + warp / (KS * NG), ks = warp % KS;
  const RowsGroup& grp = p.g[SWIGLU ? (warp / KS) % 2 : blockIdx.y];
  const bool tile_live = tile < tiles;
  const int nblk = (p.K + kBlk - 1) / kBlk;
  const int per = (nblk + KS - 1) / KS;
  const int blk0 = ks * per, blk1 = tile_live ? min(nblk, blk0 + per) : blk0;
  const int n_base = tile * 16;
  // weight rows of this lane: g and g + 8 of the tile (rows past N read row N-1 and are dropped at the end)
  const __nv_bfloat16* wrow[2];
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    const int n = max(0, min(p.N - 1, n_base + hh * 8 + g));
    wrow[hh] = grp.W + split2(n, p.N0, grp.b_s4, grp.b_s5) + t * 8 * LW;
  }
  const bool x_live = g < p.M;
  const __nv_bfloat16* xrow = p.X + (x_live ? split2(g, p.M0, p.a_s2, p.a_s3) : 0) + t * 8 * LW;
  const uint32_t my_ring = ring0 + uint32_t(warp) * (kStages * kStageBytes) + uint32_t(lane) * 16;
  auto slot = [&](int blk, int which, int piece) {
    return my_ring + uint32_t((blk - blk0) % kStages) * kStageBytes + uint32_t(which * LW + piece) * (32 * 16);
  };
  auto fill_w = [&](int blk) {
#pragma unroll
    for (int q = 0; q < LW; ++q) {
      const int k = blk * kBlk + q * 8;
      const bool ok = blk < blk1 && k + t * 8 * LW < p.K;   // K is a multiple of 8: a piece is all inside or all outside
      const int kk = ok ? k : 0;
      cp_async16(slot(blk, 0, q), wrow[0] + kk, ok);
      cp_async16(slot(blk, 1, q), wrow[1] + kk, ok);
    }
  };
  // the activations ride in the same ring (they come from L2 at best: the ring leaves little L1)
  auto fill_x = [&](int blk) {
#pragma unroll
    for (int q = 0; q < LW; ++q) {
      const int k = blk * kBlk + q * 8;
      const bool ok = x_live && blk < blk1 && k + t * 8 * LW < p.K;
      cp_async16(slot(blk, 2, q), xrow + (ok ? k : 0), ok);
    }
  };
  // the weights do not depend on the previous step: their first stages are requested before the wait
  if (p.w_const)
    for (int i = 0; i < kStages - 1; ++i) fill_w(blk0 + i);
  pdl_wait();
  for (int i = 0; i < kStages - 1; ++i) {
    if (!p.w_const) fill_w(blk0 + i);
    fill_x(blk0 + i);
    cp_async_commit();
  }
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
  for (int blk = blk0; blk < blk1; ++blk) {
    cp_async_wait<kStages - 2>();   // this lane's copies of stage `blk` have landed
    uint4 w0[LW], w1[LW], x[LW];
#pragma unroll
    for (int q = 0; q < LW; ++q) {
      w0[q] = lds128(slot(blk, 0, q));
      w1[q] = lds128(slot(blk, 1, q));
      x[q] = lds128(slot(blk, 2, q));
    }
    // refill the slot read one pass ago
    fill_w(blk + kStages - 1);
    fill_x(blk + kStages - 1);
    cp_async_commit();
#pragma unroll
    for (int q = 0; q < LW; ++q) {
      mma_bf16(acc, w0[q].x, w1[q].x, w0[q].y, w1[q].y, x[q].x, x[q].y);
      mma_bf16(acc, w0[q].z, w1[q].z, w0[q].w, w1[q].w, x[q].z, x[q].w);
    }
  }
  cp_async_wait<0>();
  // accumulator fragment: acc[0..1] = (weight row g; activation rows 2t, 2t+1), acc[2..3] = (weight row g + 8; same)
  red[warp][g][2 * t] = acc[0];
  red[warp][g][2 * t + 1] = acc[1];
  red[warp][g + 8][2 * t] = acc[2];
  red[warp][g + 8][2 * t + 1] = acc[3];
  __syncthreads();
  // thread -> (tile of the CTA, m, row of the tile) with the row fastest, so that stores to an n-contiguous C coalesce
  for (int e = threadIdx.x; e < TPC * 16 * 8; e += kWarps * 32) {
    const int nl = e % 16, m = (e / 16) % 8, tl = e / 128;
    const int n = (blockIdx.x * TPC + tl) * 16 + nl;
    if (m >= p.M || n >= p.N) continue;
    float v = 0.f;
#pragma unroll
    for (int q = 0; q < KS; ++q) v += red[tl * NG * KS + q][nl][m];
    v *= p.scale;
    if (SWIGLU) {
      float u = 0.f;
#pragma unroll
      for (int q = 0; q < KS; ++q) u += red[(tl * NG + 1) * KS + q][nl][m];
      v = silu(v) * (u * p.scale);
    }
    const RowsGroup& grp = p.g[SWIGLU ? 0 : blockIdx.y];
    if (grp.has_bias) v += __bfloat162float(grp.bias[n]);
    if (grp.act == ACT_GELU_ERF) v = gelu_erf(v);
    else if (grp.act == ACT_GELU_TANH) v = gelu_tanh(v);
    if (grp.has_res) {
      const int64_t ro = split2(m, p.M0, grp.r_s[2], grp.r_s[3]) + split2(n, p.N0, grp.r_s[4], grp.r_s[5]);
      v += grp.r_f32 ? static_cast<const float*>(grp.R)[ro] : __bfloat162float(static_cast<const __nv_bfloat16*>(grp.R)[ro]);
    }
    const int64_t co = split2(m, p.M0, grp.c_s[2], grp.c_s[3]) + split2(n, p.N0, grp.c_s[4], grp.c_s[5]);
    if (grp.c_f32) static_cast<float*>(grp.C)[co] = v;
    else static_cast<__nv_bfloat16*>(grp.C)[co] = __float2bfloat16_rn(v);
  }
}


template <int KS, int LW, int ST, bool SWIGLU>
cudaError_t launch_rows(const RowsParams& p, int tiles, int n_group, cudaStream_t st) {
  constexpr int kWarps = rows_warps(KS, SWIGLU);
  constexpr size_t smem = size_t(kWarps) * ST * 3 * LW * 32 * 16 + size_t(kWarps) * 16 * 9 * sizeof(float);
  static const cudaError_t attr =
      cudaFuncSetAttribute(gemm_rows_kernel<KS, LW, ST, SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (attr != cudaSuccess) return attr;
  constexpr int TPC = kWarps / (KS * (SWIGLU ? 2 : 1));
  dim3 grid((unsigned)((tiles + TPC - 1) / TPC), (unsigned)(SWIGLU ? 1 : n_group));
  return launch_k(gemm_rows_kernel<KS, LW, ST, SWIGLU>, grid, dim3(kWarps * 32), smem, st, p, tiles);
}

template <int LW, int ST>
cudaError_t launch_rows_ks(const RowsParams& p, int tiles, int n_group, int cps, bool swiglu, cudaStream_t st) {
  // as many warps per tile (k slices) as keep the whole launch resident at once
  const int64_t items = (int64_t)tiles * n_group, cap = 148 * kWarpsPerSm;
  (void)cps;
  if (swiglu) {
    if (items * 4 <= cap) return launch_rows<4, LW, ST, true>(p, tiles, n_group, st);
    if (items * 2 <= cap) return launch_rows<2, LW, ST, true>(p, tiles, n_group, st);
    return launch_rows<1, LW, ST, true>(p, tiles, n_group, st);
  }
  if (items * 8 <= cap) return launch_rows<8, LW, ST, false>(p, tiles, n_group, st);
  if (items * 4 <= cap) return launch_rows<4, LW, ST, false>(p, tiles, n_group, st);
  if (items * 2 <= cap) return launch_rows<2, LW, ST, false>(p, tiles, n_group, st);
  return launch_rows<1, LW, ST, false>(p, tiles, n_group, st);
}

inline bool flat(int X, int X0, int64_t s1, int64_t s0) { return X0 >= X || s1 == (int64_t)X0 * s0; }
inline bool al16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool gemm_rows_eligible(const GemmParams& g) {
  if (g.dtype != FLUID_BF16 || g.batch != 1 || g.M < 1 || g.M > 8 || g.causal != CAUSAL_NONE) return false;
  if (g.K % 8 || g.K < 8) return false;
  // both operands with a flat, contiguous k index
  if (g.a_s[5] != 1 || !flat(g.K, g.K0, g.a_s[4], 1)) return false;
  if (g.b_s[3] != 1 || !flat(g.K, g.K0, g.b_s[2], 1)) return false;
  // 16-byte loads: every row starts on a 16-byte boundary
  const int64_t rows[4] = {g.M > g.M0 ? g.a_s[2] : 0, g.M > 1 ? g.a_s[3] : 0, g.N > g.N0 ? g.b_s[4] : 0, g.N > 1 ? g.b_s[5] : 0};
  for (int64_t s : rows)
    if (s % 8) return false;
  return true;
}

cudaError_t launch_gemm_rows(const GemmParams* gs, int n_group, cudaStream_t st, int swiglu) {
  if (n_group < 1 || n_group > 3 || (swiglu && n_group != 2)) return cudaErrorInvalidValue;
  const GemmParams& g0 = gs[0];
  RowsParams p{};
  p.X = static_cast<const __nv_bfloat16*>(g0.A);
  p.M = g0.M; p.N = g0.N; p.K = g0.K; p.M0 = g0.M0; p.N0 = g0.N0;
  p.a_s2 = g0.a_s[2]; p.a_s3 = g0.a_s[3];
  p.scale = g0.scale;
  p.w_const = 1;
  if (!al16(g0.A)) return cudaErrorInvalidValue;
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
  const int tiles = (p.N + 15) / 16;
  // one 16-byte piece per lane, row and stage (wider pieces measured three times slower: a copy instruction of the
  // warp then touches every 32-byte sector half), ring five deep, which lets three CTAs share an SM
  return launch_rows_ks<1, 5>(p, tiles, n_group, 3, swiglu != 0, st);
}

}  // namespace fluid
