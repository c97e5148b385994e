// GEMM with a handful of rows (M <= 16: the LINEAR steps of single-token decoding). The step reads every
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
// roles swapped: 16 weight rows are the MMA's row operand, the activation rows its 8 columns (two MMAs side by side
// for 9 to 16 activation rows). The
// contraction index may be fed in any order as long as both operands agree, so a lane takes 8 *consecutive* k of
// one weight row (one 16-byte copy) and the same 8 k of one activation row, and two MMAs consume them: no
// unpacking, no shuffles, no exchange between lanes.
//
// A warp owns 16 weight rows and a slice of the k range; the warps that share a tile add their partial sums
// through shared memory and the CTA's threads apply bias / activation / residual and store.
// Sibling projections that share X (Q/K/V, gate/up) run as one launch (blockIdx.y = group).
#include <algorithm>

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
      if ((is_x || is_beta) && warp % wpr == 0 && lane < kXPad / 8) *reinterpret_cast<uint4*>(dst + (chunks + lane) * 8) = make_uint4(0u, 0u, 0u, 0u);
      acc = warp_sum(acc);
      if (lane == 0) part[warp] = acc;
      __syncthreads();
      if (threadIdx.x < p.M) {
        float q2 = 0.f;
        for (int q = 0; q < wpr; ++q) q2 += part[threadIdx.x * wpr + q];
        rstd[threadIdx.x] = p.gamma ? rsqrtf(q2 / p.K + p.eps) : 1.f;
      }
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

cudaError_t launch_gemm_rows(const GemmParams* gs, int n_group, cudaStream_t st, int swiglu, const RowsNorm* norm) {
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
