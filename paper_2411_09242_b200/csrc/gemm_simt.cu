// SIMT GEMM over arbitrarily strided operands (fp32 accumulate, FFMA). It serves the fp32
// configuration, whose 1e-4 tolerance rules out single-pass tf32 tensor-core products, and any
// bf16 GEMM whose layout the TMA-fed tensor-core kernel cannot express.
#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

constexpr int BM = 64, BN = 64, BK = 16;

// offset of index i split as (i / x0, i % x0); no division in the common merged case (x0 > i)
__device__ __forceinline__ int64_t split_off(int i, int x0, int64_t s1, int64_t s0) {
  if (i < x0) return (int64_t)i * s0;
  const int hi = i / x0;
  return (int64_t)hi * s1 + (int64_t)(i - hi * x0) * s0;
}

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmParams p, int a_k_fast, int b_n_fast) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN, bz = blockIdx.z;
  if (p.causal == CAUSAL_SKIP_UPPER && n0 > m0 + BM - 1) return;
  int kend = p.K;
  if (p.causal == CAUSAL_CLIP_K) kend = min(p.K, m0 + BM);
  const int64_t ab = split_off(bz, p.B0, p.a_s[0], p.a_s[1]);
  const int64_t bb = split_off(bz, p.B0, p.b_s[0], p.b_s[1]);
  const int64_t cb = split_off(bz, p.B0, p.c_s[0], p.c_s[1]);
  const T* A = static_cast<const T*>(p.A) + ab;
  const T* B = static_cast<const T*>(p.B) + bb;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  // the row / column part of each thread's four A and four B elements does not change over k
  int ar[4], akk[4], bc[4], bkk[4];
  int64_t a_row[4], b_col[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int e = tid + 256 * j;
    ar[j] = a_k_fast ? e / BK : e % BM;
    akk[j] = a_k_fast ? e % BK : e / BM;
    bc[j] = b_n_fast ? e % BN : e / BK;
    bkk[j] = b_n_fast ? e / BN : e % BK;
    a_row[j] = m0 + ar[j] < p.M ? split_off(m0 + ar[j], p.M0, p.a_s[2], p.a_s[3]) : -1;
    b_col[j] = n0 + bc[j] < p.N ? split_off(n0 + bc[j], p.N0, p.b_s[4], p.b_s[5]) : -1;
  }
  // global -> registers -> shared, with the next k-slab's loads in flight during the FFMA loop
  float va[4], vb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int k = k0 + akk[j];
      va[j] = (a_row[j] >= 0 && k < kend) ? to_f(__ldg(A + a_row[j] + split_off(k, p.K0, p.a_s[4], p.a_s[5]))) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int k = k0 + bkk[j];
      vb[j] = (b_col[j] >= 0 && k < kend) ? to_f(__ldg(B + split_off(k, p.K0, p.b_s[2], p.b_s[3]) + b_col[j])) : 0.f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < kend; k0 += BK) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      As[akk[j]][ar[j]] = va[j];
      Bs[bkk[j]][bc[j]] = vb[j];
    }
    __syncthreads();
    if (k0 + BK < kend) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  T* C = static_cast<T*>(p.C) + cb;
  float* Cf = static_cast<float*>(p.C) + cb;
  const int64_t rb = p.has_res ? split_off(bz, p.B0, p.r_s[0], p.r_s[1]) : 0;
  const T* R = p.has_res ? static_cast<const T*>(p.R) + rb : nullptr;
  const float* Rf = static_cast<const float*>(p.R) + rb;
  const bool c_wide = p.c_f32 && sizeof(T) == 2, r_wide = p.r_f32 && sizeof(T) == 2;
  const T* bias = static_cast<const T*>(p.bias);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
    const int64_t cm = split_off(m, p.M0, p.c_s[2], p.c_s[3]);
    const int64_t rm = R ? split_off(m, p.M0, p.r_s[2], p.r_s[3]) : 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= p.N) continue;
      float v = acc[i][j] * p.scale;
      if (p.has_bias) v += to_f(bias[n]);
      if (p.act == ACT_GELU_ERF) v = gelu_erf(v);
      else if (p.act == ACT_GELU_TANH) v = gelu_tanh(v);
      if (R) {
        const int64_t ro = rm + split_off(n, p.N0, p.r_s[4], p.r_s[5]);
        v += r_wide ? Rf[ro] : to_f(R[ro]);
      }
      const int64_t co = cm + split_off(n, p.N0, p.c_s[4], p.c_s[5]);
      if (c_wide) Cf[co] = v;
      else C[co] = from_f<T>(v);
    }
  }
}

// Small products (the fp32 toy configuration: 32 rows, 128-512 columns): the tiled kernel above would run as two to
// eight CTAs, each a serial loop of load -> shared memory -> barrier -> FFMA over k with one slab in flight (15-26 us a
// launch). Here a CTA owns one output row and 32 columns: its eight warps split the k range (lane = column: A's element
// is one broadcast load, B's row of 32 a coalesced one, eight of each in flight per thread), the partial sums meet in
// shared memory and are added in warp order. A hundred CTAs or more, one barrier.
template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_small_kernel(GemmParams p) {
  __shared__ float part[8][32];
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * 32 + lane, m = blockIdx.y, bz = blockIdx.z;
  const bool col_ok = n < p.N && !(p.causal == CAUSAL_SKIP_UPPER && n > (m / BM) * BM + BM - 1);
  int kend = p.K;
  if (p.causal == CAUSAL_CLIP_K) kend = min(p.K, (m / BM) * BM + BM);
  const int per = ((kend + 7) / 8 + 7) & ~7;          // k elements per warp, a multiple of the unroll
  const int k0 = warp * per, k1 = min(kend, k0 + per);
  const T* A = static_cast<const T*>(p.A) + split_off(bz, p.B0, p.a_s[0], p.a_s[1]) + split_off(m, p.M0, p.a_s[2], p.a_s[3]);
  const T* B = static_cast<const T*>(p.B) + split_off(bz, p.B0, p.b_s[0], p.b_s[1]) + (col_ok ? split_off(n, p.N0, p.b_s[4], p.b_s[5]) : 0);
  pdl_wait();
  float acc = 0.f;
  if (col_ok) {
    int k = k0;
    for (; k + 8 <= k1; k += 8) {
      float a[8], b[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        a[u] = to_f(__ldg(A + split_off(k + u, p.K0, p.a_s[4], p.a_s[5])));
        b[u] = to_f(__ldg(B + split_off(k + u, p.K0, p.b_s[2], p.b_s[3])));
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) acc = fmaf(a[u], b[u], acc);
    }
    for (; k < k1; ++k)
      acc = fmaf(to_f(__ldg(A + split_off(k, p.K0, p.a_s[4], p.a_s[5]))), to_f(__ldg(B + split_off(k, p.K0, p.b_s[2], p.b_s[3]))), acc);
  }
  part[warp][lane] = acc;
  __syncthreads();
  if (warp != 0 || !col_ok) return;
  float v = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) v += part[w][lane];
  v *= p.scale;
  if (p.has_bias) v += to_f(static_cast<const T*>(p.bias)[n]);
  if (p.act == ACT_GELU_ERF) v = gelu_erf(v);
  else if (p.act == ACT_GELU_TANH) v = gelu_tanh(v);
  if (p.has_res) {
    const int64_t ro = split_off(bz, p.B0, p.r_s[0], p.r_s[1]) + split_off(m, p.M0, p.r_s[2], p.r_s[3]) + split_off(n, p.N0, p.r_s[4], p.r_s[5]);
    v += (p.r_f32 && sizeof(T) == 2) ? static_cast<const float*>(p.R)[ro] : to_f(static_cast<const T*>(p.R)[ro]);
  }
  const int64_t co = split_off(bz, p.B0, p.c_s[0], p.c_s[1]) + split_off(m, p.M0, p.c_s[2], p.c_s[3]) + split_off(n, p.N0, p.c_s[4], p.c_s[5]);
  if (p.c_f32 && sizeof(T) == 2) static_cast<float*>(p.C)[co] = v;
  else static_cast<T*>(p.C)[co] = from_f<T>(v);
}

cudaError_t launch_gemm_simt(const GemmParams& p, cudaStream_t st) {
  dim3 grid((p.N + BN - 1) / BN, (p.M + BM - 1) / BM, p.batch);
  // few tiles (and few enough rows for a CTA per row and 32 columns to stay a modest grid): the small form
  if ((int64_t)grid.x * grid.y * grid.z <= 32 && (int64_t)p.M * ((p.N + 31) / 32) * p.batch <= 4096) {
    dim3 small((p.N + 31) / 32, p.M, p.batch);
    return p.dtype == FLUID_BF16 ? launch_k(gemm_simt_small_kernel<__nv_bfloat16>, small, 256, 0, st, p)
                                 : launch_k(gemm_simt_small_kernel<float>, small, 256, 0, st, p);
  }
  const int a_k_fast = p.a_s[5] == 1 || p.a_s[3] != 1;
  const int b_n_fast = p.b_s[5] == 1 || p.b_s[3] != 1;
  return p.dtype == FLUID_BF16 ? launch_k(gemm_simt_kernel<__nv_bfloat16>, grid, 256, 0, st, p, a_k_fast, b_n_fast)
                               : launch_k(gemm_simt_kernel<float>, grid, 256, 0, st, p, a_k_fast, b_n_fast);
}

}  // namespace fluid
