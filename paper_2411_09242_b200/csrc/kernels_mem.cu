// Memory-bound kernels: embedding gather, LayerNorm/RMSNorm (+ fused residual), softmax
// (scale + causal mask), rotary embedding, elementwise ops, layout transforms. All move
// 16-byte vectors where shapes allow and keep their arithmetic in fp32.
#include <algorithm>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// ---- EMBED: y[t, :] = tok[ids[t], :] (+ pos[t % S, :]) -------------------------------------------
template <typename T, bool VECTOR>
__global__ void embed_kernel(EmbedParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.x;
  int id = p.ids[t];
  id = min(max(id, 0), p.V - 1);
  const T* tok = static_cast<const T*>(p.tok) + (size_t)id * p.H;
  int prow = t % p.S;
  if (p.pos_off) prow = min(max(prow + p.pos_off[(t / p.S) * p.pos_off_stride], 0), p.P - 1);
  const T* pos = p.pos ? static_cast<const T*>(p.pos) + (size_t)prow * p.H : nullptr;
  T* y = static_cast<T*>(p.y) + (size_t)t * p.H;
  float* yf = static_cast<float*>(p.y) + (size_t)t * p.H;
  const bool wide = p.y_f32 && sizeof(T) == 2;
  if (VECTOR) {
    constexpr int V = VecOf<T>::N;
    for (int c = threadIdx.x * V; c < p.H; c += blockDim.x * V) {
      float a[V];
      load16(tok + c, a);
      if (pos) {
        float b[V];
        load16(pos + c, b);
#pragma unroll
        for (int i = 0; i < V; ++i) a[i] += b[i];
      }
      if (wide) {
#pragma unroll
        for (int i = 0; i < V; i += 4)
          *reinterpret_cast<float4*>(yf + c + i) = make_float4(a[i], a[i + 1], a[i + 2], a[i + 3]);
      } else {
        store16(y + c, a);
      }
    }
  } else {
    for (int c = threadIdx.x; c < p.H; c += blockDim.x) {
      float a = to_f(tok[c]);
      if (pos) a += to_f(pos[c]);
      if (wide) yf[c] = a;
      else y[c] = from_f<T>(a);
    }
  }
}

template <typename T>
static cudaError_t embed_t(const EmbedParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.H % V == 0 && aligned16(p.tok) && aligned16(p.y) && (!p.pos || aligned16(p.pos));
  const int threads = std::min(256, std::max(32, ((p.H / (vec ? V : 1)) + 31) / 32 * 32));
  return vec ? launch_k(embed_kernel<T, true>, p.tokens, threads, 0, st, p) : launch_k(embed_kernel<T, false>, p.tokens, threads, 0, st, p);
}

cudaError_t launch_embed(const EmbedParams& p, cudaStream_t st) {
  return p.dtype == FLUID_BF16 ? embed_t<__nv_bfloat16>(p, st) : embed_t<float>(p, st);
}

// ---- NORM: one row per CTA, row cached in registers, two block reductions ------------------------
// In bf16 models the input, the residual addend and one copy of the output may be fp32: the
// residual stream is carried in fp32 so that rounding does not pile up layer after layer.
constexpr int NORM_MAXC = 4;

template <typename T, int V>
__device__ __forceinline__ void norm_load(const void* base, bool f32, size_t row_off, int c, float (&a)[V]) {
  if (V == 1) {
    a[0] = f32 ? static_cast<const float*>(base)[row_off + c] : to_f(static_cast<const T*>(base)[row_off + c]);
  } else if (f32 || sizeof(T) == 4) {
    const float* q = static_cast<const float*>(base) + row_off + (size_t)c * V;
#pragma unroll
    for (int i = 0; i < V; i += 4) {
      const float4 f = *reinterpret_cast<const float4*>(q + i);
      a[i] = f.x; a[i + 1] = f.y; a[i + 2] = f.z; a[i + 3] = f.w;
    }
  } else {
    float t8[VecOf<T>::N];
    load16(static_cast<const T*>(base) + row_off + (size_t)c * V, t8);
#pragma unroll
    for (int i = 0; i < V; ++i) a[i] = t8[i];
  }
}

template <typename T, bool VECTOR>
__global__ void norm_kernel(NormParams p) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int V = VECTOR ? VecOf<T>::N : 1;
  __shared__ float red[32];
  const size_t roff = (size_t)blockIdx.x * p.width;
  const T* gamma = static_cast<const T*>(p.gamma);
  const T* beta = static_cast<const T*>(p.beta);
  const int nch = p.width / V;
  float v[NORM_MAXC][V];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < NORM_MAXC; ++j) {
    const int c = threadIdx.x + j * blockDim.x;
    if (c < nch) {
      norm_load<T, V>(p.x, p.x_f32, roff, c, v[j]);
      if (p.res) {
        float b[V];
        norm_load<T, V>(p.res, p.res_f32, roff, c, b);
#pragma unroll
        for (int i = 0; i < V; ++i) v[j][i] += b[i];
      }
#pragma unroll
      for (int i = 0; i < V; ++i) s += p.rms ? v[j][i] * v[j][i] : v[j][i];
    }
  }
  s = block_sum(s, red);
  float mean = 0.f, rstd;
  if (p.rms) {
    rstd = rsqrtf(s / p.width + p.eps);
  } else {
    mean = s / p.width;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < NORM_MAXC; ++j) {
      const int c = threadIdx.x + j * blockDim.x;
      if (c < nch) {
#pragma unroll
        for (int i = 0; i < V; ++i) q += (v[j][i] - mean) * (v[j][i] - mean);
      }
    }
    q = block_sum(q, red);
    rstd = rsqrtf(q / p.width + p.eps);
  }
  T* y_lo = static_cast<T*>(p.y_lo);
#pragma unroll
  for (int j = 0; j < NORM_MAXC; ++j) {
    const int c = threadIdx.x + j * blockDim.x;
    if (c < nch) {
      float g[V], b[V], o[V];
      norm_load<T, V>(gamma, false, 0, c, g);
      if (beta) norm_load<T, V>(beta, false, 0, c, b);
#pragma unroll
      for (int i = 0; i < V; ++i) o[i] = (v[j][i] - mean) * rstd * g[i] + (beta ? b[i] : 0.f);
      if (VECTOR) {
        if (y_lo) {
          float t8[VecOf<T>::N];
#pragma unroll
          for (int i = 0; i < V; ++i) t8[i] = o[i];
          store16(y_lo + roff + (size_t)c * V, t8);
        }
        if (p.y_hi) {
#pragma unroll
          for (int i = 0; i < V; i += 4)
            *reinterpret_cast<float4*>(p.y_hi + roff + (size_t)c * V + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
        }
      } else {
        if (y_lo) y_lo[roff + c] = from_f<T>(o[0]);
        if (p.y_hi) p.y_hi[roff + c] = o[0];
      }
    }
  }
}

// Row handled by WPR warps (1, 2, 4 or 8) of a 256-thread CTA: each lane owns NCH 16-byte
// chunks; sums go through shuffles and, for WPR > 1, a few words of shared memory.
template <int WPR>
__device__ __forceinline__ float row_sum(float v, float* red, int warp, int lane) {
  v = warp_sum(v);
  if (WPR == 1) return v;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = 0.f;
  const int g0 = warp / WPR * WPR;
#pragma unroll
  for (int i = 0; i < WPR; ++i) t += red[g0 + i];
  return t;
}

// EARLY: the gain and bias are read into registers before the wait for the previous step (short grids are
// latency-bound and win from the overlap; long grids are bandwidth-bound and want the registers for occupancy).
template <typename T, int NCH, int WPR, bool EARLY>
__global__ void __launch_bounds__(256, (!EARLY && NCH <= 3) ? 5 : 1) norm_warp_kernel(NormParams p) {
  pdl_launch_dependents();
  constexpr int V = VecOf<T>::N;
  __shared__ float red[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * (8 / WPR) + warp / WPR;
  const bool live = row < p.rows;
  const size_t roff = (size_t)(live ? row : 0) * p.width;
  const int nch = live ? p.width / V : 0;
  const int c_first = (warp % WPR) * 32 + lane;
  // gain and bias are constants of the plan, not outputs of the previous step: they are fetched while
  // that step is still finishing
  const T* gamma = static_cast<const T*>(p.gamma);
  const T* beta = static_cast<const T*>(p.beta);
  float gv[EARLY ? NCH : 1][V], bv[EARLY ? NCH : 1][V];
  if (EARLY) {
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int c = c_first + 32 * WPR * j;
#pragma unroll
      for (int i = 0; i < V; ++i) bv[j][i] = 0.f;
      if (c < nch) {
        norm_load<T, V>(gamma, false, 0, c, gv[j]);
        if (beta) norm_load<T, V>(beta, false, 0, c, bv[j]);
      }
    }
  }
  pdl_wait();
  float v[NCH][V];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int c = c_first + 32 * WPR * j;
    if (c < nch) norm_load<T, V>(p.x, p.x_f32, roff, c, v[j]);
  }
  if (p.res) {
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int c = c_first + 32 * WPR * j;
      if (c < nch) {
        float b[V];
        norm_load<T, V>(p.res, p.res_f32, roff, c, b);
#pragma unroll
        for (int i = 0; i < V; ++i) v[j][i] += b[i];
      }
    }
  }
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    if (c_first + 32 * WPR * j < nch) {
#pragma unroll
      for (int i = 0; i < V; ++i) s += p.rms ? v[j][i] * v[j][i] : v[j][i];
    }
  }
  s = row_sum<WPR>(s, red, warp, lane);
  float mean = 0.f, rstd;
  if (p.rms) {
    rstd = rsqrtf(s / p.width + p.eps);
  } else {
    mean = s / p.width;
    float q = 0.f;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      if (c_first + 32 * WPR * j < nch) {
#pragma unroll
        for (int i = 0; i < V; ++i) q += (v[j][i] - mean) * (v[j][i] - mean);
      }
    }
    q = row_sum<WPR>(q, red, warp, lane);
    rstd = rsqrtf(q / p.width + p.eps);
  }
  T* y_lo = static_cast<T*>(p.y_lo);
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int c = c_first + 32 * WPR * j;
    if (c < nch) {
      float o[V];
      if (EARLY) {
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = (v[j][i] - mean) * rstd * gv[j][i] + bv[j][i];
      } else {
        float g[V], b[V];
        norm_load<T, V>(gamma, false, 0, c, g);
        if (beta) norm_load<T, V>(beta, false, 0, c, b);
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = (v[j][i] - mean) * rstd * g[i] + (beta ? b[i] : 0.f);
      }
      if (y_lo) {
        float t8[VecOf<T>::N];
#pragma unroll
        for (int i = 0; i < V; ++i) t8[i] = o[i];
        store16(y_lo + roff + (size_t)c * V, t8);
      }
      if (p.y_hi) {
#pragma unroll
        for (int i = 0; i < V; i += 4)
          *reinterpret_cast<float4*>(p.y_hi + roff + (size_t)c * V + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
      }
    }
  }
}

// Long inputs (many more rows than resident warps): persistent warps, each walking rows with the grid's stride. The
// row's 16-byte pieces reach the lane that will use them through a lane-private ring of asynchronous copies in
// shared memory (no barrier: a lane reads back only what it copied), so a warp has RING - 1 rows in flight while it
// reduces and stores one, and the gain and bias are read once per warp instead of once per row.
constexpr int NORM_RING = 4;
__device__ __forceinline__ void norm_cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// sum over the WPR warps that share a row (named barrier per row group; `red` alternates between two sets of slots
// so that a fast warp's next sum cannot overwrite what a slow warp has not read yet)
template <int WPR>
__device__ __forceinline__ float ring_row_sum(float v, float* red, int slot, int warp, int lane) {
  v = warp_sum(v);
  if (WPR == 1) return v;
  if (lane == 0) red[slot * 8 + warp] = v;
  asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / WPR), "r"(WPR * 32) : "memory");
  float t = 0.f;
  const int g0 = warp / WPR * WPR;
#pragma unroll
  for (int i = 0; i < WPR; ++i) t += red[slot * 8 + g0 + i];
  return t;
}

template <typename T, int NCH, int WPR, bool XF32>
__global__ void __launch_bounds__(256, 2) norm_ring_kernel(NormParams p) {
  __shared__ float red[4 * 8];
  constexpr int V = VecOf<T>::N;                      // elements per chunk (a lane's unit of work)
  constexpr int PCS = (XF32 && sizeof(T) == 2) ? 2 : 1;   // 16-byte pieces per chunk in the ring
  constexpr int SLOT = NCH * PCS * 512;               // bytes per row and warp
  extern __shared__ __align__(16) unsigned char norm_ring_raw[];
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nch = p.width / V;
  const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(norm_ring_raw)) + uint32_t(warp) * (NORM_RING * SLOT) + uint32_t(lane) * 16;
  const T* gamma = static_cast<const T*>(p.gamma);
  const T* beta = static_cast<const T*>(p.beta);
  const int c_first = (warp % WPR) * 32 + lane;
  float gv[NCH][V], bv[NCH][V];
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int c = c_first + 32 * WPR * j;
#pragma unroll
    for (int i = 0; i < V; ++i) { gv[j][i] = 0.f; bv[j][i] = 0.f; }
    if (c < nch) {
      norm_load<T, V>(gamma, false, 0, c, gv[j]);
      if (beta) norm_load<T, V>(beta, false, 0, c, bv[j]);
    }
  }
  constexpr int RPB = 8 / WPR;   // rows per CTA and pass
  const int64_t stride = (int64_t)gridDim.x * RPB;
  const int64_t row0 = (int64_t)blockIdx.x * RPB + warp / WPR;
  const int64_t n_mine = row0 < p.rows ? (p.rows - row0 + stride - 1) / stride : 0;
  auto fill = [&](int64_t i) {
    if (i >= n_mine) return;
    const size_t roff = (size_t)(row0 + i * stride) * p.width;
    const uint32_t dst = ring + uint32_t(i % NORM_RING) * SLOT;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int c = c_first + 32 * WPR * j;
      if (c < nch) {
        if (PCS == 2) {
          const float* src = static_cast<const float*>(p.x) + roff + (size_t)c * V;
          norm_cp16(dst + (2 * j) * 512, src);
          norm_cp16(dst + (2 * j + 1) * 512, src + 4);
        } else {
          norm_cp16(dst + j * 512, static_cast<const unsigned char*>(p.x) + (roff + (size_t)c * V) * (XF32 ? 4 : sizeof(T)));
        }
      }
    }
  };
  pdl_wait();
  for (int i = 0; i < NORM_RING - 1; ++i) {
    fill(i);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  T* y_lo = static_cast<T*>(p.y_lo);
#pragma unroll 1
  for (int64_t i = 0; i < n_mine; ++i) {
    asm volatile("cp.async.wait_group %0;" ::"n"(NORM_RING - 2) : "memory");
    const uint32_t src = ring + uint32_t(i % NORM_RING) * SLOT;
    float v[NCH][V];
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int c = c_first + 32 * WPR * j;
#pragma unroll
      for (int q = 0; q < V; ++q) v[j][q] = 0.f;
      if (c < nch) {
        if (XF32 || sizeof(T) == 4) {
#pragma unroll
          for (int h = 0; h < PCS; ++h) {
            uint4 w;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(src + (PCS * j + h) * 512) : "memory");
            v[j][4 * h] = __uint_as_float(w.x); v[j][4 * h + 1] = __uint_as_float(w.y);
            v[j][4 * h + 2] = __uint_as_float(w.z); v[j][4 * h + 3] = __uint_as_float(w.w);
          }
        } else {
          uint4 w;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(src + j * 512) : "memory");
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            v[j][2 * q] = __uint_as_float(ww[q] << 16);
            v[j][2 * q + 1] = __uint_as_float(ww[q] & 0xffff0000u);
          }
        }
#pragma unroll
        for (int q = 0; q < V; ++q) s += p.rms ? v[j][q] * v[j][q] : v[j][q];
      }
    }
    fill(i + NORM_RING - 1);   // refills the slot read one pass ago
    asm volatile("cp.async.commit_group;" ::: "memory");
    const int par = int(i & 1) * 2;
    s = ring_row_sum<WPR>(s, red, par, warp, lane);
    float mean = 0.f, rstd;
    if (p.rms) {
      rstd = rsqrtf(s / p.width + p.eps);
    } else {
      mean = s / p.width;
      float q2 = 0.f;
#pragma unroll
      for (int j = 0; j < NCH; ++j)
        if (c_first + 32 * WPR * j < nch) {
#pragma unroll
          for (int q = 0; q < V; ++q) q2 += (v[j][q] - mean) * (v[j][q] - mean);
        }
      q2 = ring_row_sum<WPR>(q2, red, par + 1, warp, lane);
      rstd = rsqrtf(q2 / p.width + p.eps);
    }
    const size_t roff = (size_t)(row0 + i * stride) * p.width;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int c = c_first + 32 * WPR * j;
      if (c < nch) {
        float o[V];
#pragma unroll
        for (int q = 0; q < V; ++q) o[q] = (v[j][q] - mean) * rstd * gv[j][q] + bv[j][q];
        if (y_lo) {
          float t8[VecOf<T>::N];
#pragma unroll
          for (int q = 0; q < V; ++q) t8[q] = o[q];
          store16(y_lo + roff + (size_t)c * V, t8);
        }
        if (p.y_hi) {
#pragma unroll
          for (int q = 0; q < V; q += 4)
            *reinterpret_cast<float4*>(p.y_hi + roff + (size_t)c * V + q) = make_float4(o[q], o[q + 1], o[q + 2], o[q + 3]);
        }
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <typename T, int NCH, int WPR, bool XF32>
static cudaError_t norm_ring_launch(const NormParams& p, cudaStream_t st) {
  constexpr int PCS = (XF32 && sizeof(T) == 2) ? 2 : 1;
  constexpr int smem = 8 * NORM_RING * NCH * PCS * 512;
  static const cudaError_t attr = cudaFuncSetAttribute(norm_ring_kernel<T, NCH, WPR, XF32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (attr != cudaSuccess) return attr;
  const int per_sm = std::max(1, std::min(2, (200 * 1024) / smem));   // two CTAs per SM by registers
  return launch_k(norm_ring_kernel<T, NCH, WPR, XF32>, 148u * per_sm, 256, smem, st, p);
}

template <typename T>
static cudaError_t norm_t(const NormParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.width % V == 0 && aligned16(p.x) && (!p.y_lo || aligned16(p.y_lo)) && (!p.y_hi || aligned16(p.y_hi)) &&
                   aligned16(p.gamma) && (!p.beta || aligned16(p.beta)) && (!p.res || aligned16(p.res));
  const int nch = p.width / (vec ? V : 1);
  if (vec && nch <= 32 * 8 * 4) {
    // warps per row so that a lane owns at most 4 chunks
    int wpr = nch <= 128 ? 1 : (nch <= 256 ? 2 : (nch <= 512 ? 4 : 8));
    // few rows (a 128-token encoder): the launch is one dependent chain of latencies, and a row spread over more warps
    // and the rows over more SMs shortens it (128 x 768: 2.7 us a launch with one warp per row on 16 SMs, 1.9 us with a
    // CTA per row on 128), as long as the grid stays one CTA per SM and a warp still has a quarter of its lanes busy
    while (wpr < 8 && (int64_t)p.rows * (2 * wpr) <= 148 * 8 && nch >= 8 * (2 * wpr)) wpr *= 2;
    const int per_lane = (nch + 32 * wpr - 1) / (32 * wpr);
    const unsigned grid = (unsigned)((p.rows + 8 / wpr - 1) / (8 / wpr));
    // (up to four CTAs' worth of rows per SM: 4096 x 768 runs 0.4 us a launch shorter inside a plan with the constants
    // fetched ahead, although its 112 registers make it two waves where the late form is one)
    const bool early = grid <= 148u * 4u;
    // many more rows than resident warps, no second addend: the persistent ring kernel
    // (with fewer rows per warp the ring never fills: measured slower on the 2048- and 4096-row norms of the model steps)
    if (!p.res && (int64_t)p.rows * wpr >= 148 * 2 * 8 * 8 && (sizeof(T) == 2 || !p.x_f32)) {
      const bool xf = p.x_f32 && sizeof(T) == 2;
#define NR_LAUNCH(N, W) return xf ? norm_ring_launch<T, N, W, true>(p, st) : norm_ring_launch<T, N, W, false>(p, st)
#define NR_PICK(W)                  \
  if (per_lane <= 1) NR_LAUNCH(1, W); \
  if (per_lane <= 2) NR_LAUNCH(2, W); \
  if (per_lane <= 3) NR_LAUNCH(3, W); \
  NR_LAUNCH(4, W)
      if (wpr == 1) { NR_PICK(1); }
      if (wpr == 2) { NR_PICK(2); }
      if (wpr == 4) { NR_PICK(4); }
      NR_PICK(8);
#undef NR_PICK
#undef NR_LAUNCH
    }
#define NW_LAUNCH(N, W) return early ? launch_k(norm_warp_kernel<T, N, W, true>, grid, 256, 0, st, p) \
                                     : launch_k(norm_warp_kernel<T, N, W, false>, grid, 256, 0, st, p)
#define NW_PICK(W)              \
  if (per_lane <= 1) NW_LAUNCH(1, W); \
  if (per_lane <= 2) NW_LAUNCH(2, W); \
  if (per_lane <= 3) NW_LAUNCH(3, W); \
  NW_LAUNCH(4, W)
    if (wpr == 1) { NW_PICK(1); }
    if (wpr == 2) { NW_PICK(2); }
    if (wpr == 4) { NW_PICK(4); }
    NW_PICK(8);
#undef NW_PICK
#undef NW_LAUNCH
  }
  int threads = (nch + 31) / 32 * 32;
  threads = std::min(1024, std::max(32, threads));
  if ((int64_t)threads * NORM_MAXC < nch) return cudaErrorInvalidValue;  // rejected at plan time
  return vec ? launch_k(norm_kernel<T, true>, p.rows, threads, 0, st, p) : launch_k(norm_kernel<T, false>, p.rows, threads, 0, st, p);
}

cudaError_t launch_norm(const NormParams& p, cudaStream_t st) {
  return p.dtype == FLUID_BF16 ? norm_t<__nv_bfloat16>(p, st) : norm_t<float>(p, st);
}

// ---- SOFTMAX: one warp per row, the row held in registers -----------------------------------------
template <typename T>
__device__ __forceinline__ float sm_exp(float x) {
  return sizeof(T) == 2 ? __expf(x) : expf(x);
}

template <typename T, int NCH, bool VECTOR>
__global__ void softmax_warp_kernel(SoftmaxParams p) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int V = VECTOR ? VecOf<T>::N : 1;
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const T* x = static_cast<const T*>(p.x) + row * p.n;
  T* y = static_cast<T*>(p.y) + row * p.n;
  const int valid = p.causal ? min(p.n, int(row % p.rows_per_mat) + 1) : p.n;
  float v[NCH][V];
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int base = (lane + 32 * j) * V;
    if (base < valid) {
      if (VECTOR) {
        float a[VecOf<T>::N];
        load16(x + base, a);
#pragma unroll
        for (int i = 0; i < V; ++i) v[j][i] = (base + i < valid) ? a[i] * p.scale : -INFINITY;
      } else {
        v[j][0] = to_f(x[base]) * p.scale;
      }
#pragma unroll
      for (int i = 0; i < V; ++i) m = fmaxf(m, v[j][i]);
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i) v[j][i] = -INFINITY;
    }
  }
  m = warp_max(m);
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
#pragma unroll
    for (int i = 0; i < V; ++i) {
      v[j][i] = sm_exp<T>(v[j][i] - m);  // exp(-inf) = 0 for masked entries
      s += v[j][i];
    }
  }
  s = warp_sum(s);
  const float inv = 1.f / s;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int base = (lane + 32 * j) * V;
    if (base < p.n) {
      if (VECTOR) {
        float o[VecOf<T>::N];
#pragma unroll
        for (int i = 0; i < V; ++i) o[i] = v[j][i] * inv;
        store16(y + base, o);
      } else {
        y[base] = from_f<T>(v[j][0] * inv);
      }
    }
  }
}

// bf16 rows kept packed in registers (16 bytes per chunk): exp is evaluated twice (sum, then
// output) so that twice as many rows are in flight per SM. CAUSAL adds the per-row bounds;
// the dense instantiation carries no per-element predicates at all.
template <int NCH, bool CAUSAL>
__global__ void __launch_bounds__(256) softmax_bf16_kernel(SoftmaxParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(p.x) + row * p.n;
  __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.y) + row * p.n;
  const int valid = CAUSAL ? min(p.n, int(row % p.rows_per_mat) + 1) : p.n;
  const int write_end = (CAUSAL && p.zero_block > 0) ? min(p.n, (valid + p.zero_block - 1) / p.zero_block * p.zero_block) : p.n;
  const float k = p.scale * 1.4426950408889634f;  // exp(x) = exp2(x * log2 e)
  // Columns past `valid` (and past the row's end) are set to -inf once, right after the load: they
  // then drop out of max and sum and come out as exact zeros with no further predicates.
  constexpr uint32_t NEG2 = 0xFF80FF80u;  // two bf16 -inf
  uint4 raw[NCH];
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int base = (lane + 32 * j) * 8;
    raw[j] = base < valid ? *reinterpret_cast<const uint4*>(x + base) : make_uint4(NEG2, NEG2, NEG2, NEG2);
  }
  // (a separate loop: every load above is in flight before the first fix-up touches its data)
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int base = (lane + 32 * j) * 8;
    if (CAUSAL && base < valid && base + 8 > valid) {
      uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (base + 2 * i >= valid) w[i] = NEG2;
        else if (base + 2 * i + 1 >= valid) w[i] = (w[i] & 0xffffu) | 0xFF800000u;
      }
      raw[j] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
  float m = -INFINITY;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      m = fmaxf(m, fmaxf(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)));
  }
  m = warp_max(m) * k;  // k > 0: max commutes with the scaling
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      s += exp2f(fmaf(__uint_as_float(w[i] << 16), k, -m)) + exp2f(fmaf(__uint_as_float(w[i] & 0xffff0000u), k, -m));
  }
  s = warp_sum(s);
  const float inv = 1.f / s;
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int base = (lane + 32 * j) * 8;
    if (base < write_end) {
      const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
      uint32_t q[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        q[i] = pack_bf16x2(exp2f(fmaf(__uint_as_float(w[i] << 16), k, -m)) * inv,
                           exp2f(fmaf(__uint_as_float(w[i] & 0xffff0000u), k, -m)) * inv);
      *reinterpret_cast<uint4*>(y + base) = make_uint4(q[0], q[1], q[2], q[3]);
    }
  }
}

// Fallback for rows too long for the register-resident kernel: one CTA per row, three sweeps.
template <typename T>
__global__ void softmax_block_kernel(SoftmaxParams p) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float red[32];
  const int64_t row = blockIdx.x;
  const T* x = static_cast<const T*>(p.x) + row * p.n;
  T* y = static_cast<T*>(p.y) + row * p.n;
  const int valid = p.causal ? min(p.n, int(row % p.rows_per_mat) + 1) : p.n;
  float m = -INFINITY;
  for (int c = threadIdx.x; c < valid; c += blockDim.x) m = fmaxf(m, to_f(x[c]) * p.scale);
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = (threadIdx.x & 31) < (blockDim.x >> 5) ? red[threadIdx.x & 31] : -INFINITY;
  m = warp_max(m);
  float s = 0.f;
  for (int c = threadIdx.x; c < valid; c += blockDim.x) s += expf(to_f(x[c]) * p.scale - m);
  s = block_sum(s, red);
  const float inv = 1.f / s;
  for (int c = threadIdx.x; c < p.n; c += blockDim.x)
    y[c] = from_f<T>(c < valid ? expf(to_f(x[c]) * p.scale - m) * inv : 0.f);
}

template <typename T>
static cudaError_t softmax_t(const SoftmaxParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.n % V == 0 && aligned16(p.x) && aligned16(p.y);
  const int per_lane = (p.n + 32 * (vec ? V : 1) - 1) / (32 * (vec ? V : 1));
  if (sizeof(T) == 2 && vec && per_lane <= 16 && p.scale > 0.f) {
    const int w8 = 8;
    const unsigned g8 = (unsigned)((p.rows + w8 - 1) / w8);
#define SB_LAUNCH(N)                                                                           \
  return p.causal ? launch_k(softmax_bf16_kernel<N, true>, g8, w8 * 32, 0, st, p)              \
                  : launch_k(softmax_bf16_kernel<N, false>, g8, w8 * 32, 0, st, p)
    if (per_lane <= 1) SB_LAUNCH(1);
    if (per_lane <= 2) SB_LAUNCH(2);
    if (per_lane <= 4) SB_LAUNCH(4);
    if (per_lane <= 8) SB_LAUNCH(8);
    SB_LAUNCH(16);
#undef SB_LAUNCH
  }
  const int warps = 4;
  const unsigned grid = (unsigned)((p.rows + warps - 1) / warps);
#define SM_LAUNCH(NCH, VEC) return launch_k(softmax_warp_kernel<T, NCH, VEC>, grid, warps * 32, 0, st, p)
  if (vec && per_lane <= 1) SM_LAUNCH(1, true);
  else if (vec && per_lane <= 2) SM_LAUNCH(2, true);
  else if (vec && per_lane <= 4) SM_LAUNCH(4, true);
  else if (vec && per_lane <= 8) SM_LAUNCH(8, true);
  else if (vec && per_lane <= 16 && sizeof(T) == 4) SM_LAUNCH(16, true);
  else if (!vec && per_lane <= 8) SM_LAUNCH(8, false);
  else return launch_k(softmax_block_kernel<T>, (unsigned)p.rows, 256, 0, st, p);
#undef SM_LAUNCH
}

cudaError_t launch_softmax(const SoftmaxParams& p, cudaStream_t st) {
  return p.dtype == FLUID_BF16 ? softmax_t<__nv_bfloat16>(p, st) : softmax_t<float>(p, st);
}

// ---- ROPE: one thread per rotated pair, threads ordered as the tensor lies in memory --------------
template <typename T>
__global__ void rope_kernel(RopeParams p, int64_t total) {
  pdl_launch_dependents();
  pdl_wait();
  const int half = p.dims[3] / 2;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int idx[4];
    int64_t rem = i;
#pragma unroll
    for (int k = 3; k >= 0; --k) {
      const int d = p.order[k];
      const int ext = d == 3 ? half : p.dims[d];
      idx[d] = int(rem % ext);
      rem /= ext;
    }
    const int pr = idx[3];
    const int d0 = p.interleaved ? 2 * pr : pr, d1 = p.interleaved ? 2 * pr + 1 : pr + half;
    const int64_t base = idx[0] * p.st[0] + idx[1] * p.st[1] + idx[2] * p.st[2];
    float sn, cs;
    const int pos0 = p.pos ? p.pos[idx[0] * p.pos_stride] : 0;
    float fh, fl;
    rope_freq(p.freq, pr, p.dims[3], fh, fl);
    rope_sincos(idx[1] + pos0, fh, fl, sn, cs);
    const T* x = static_cast<const T*>(p.x);
    T* y = static_cast<T*>(p.y);
    const float a = to_f(x[base + d0 * p.st[3]]), b = to_f(x[base + d1 * p.st[3]]);
    y[base + d0 * p.st[3]] = from_f<T>(a * cs - b * sn);
    y[base + d1 * p.st[3]] = from_f<T>(b * cs + a * sn);
  }
}

// Vector variant (D contiguous, rotate-half pairing, bf16): a thread owns 8 pairs of one token
// and applies the same 8 (cos, sin) to a group of heads, moving 16 bytes per access.
constexpr int ROPE_HG = 4;
__global__ void __launch_bounds__(256) rope_vec_kernel(RopeParams p, int64_t total, int hgroups) {
  pdl_launch_dependents();
  pdl_wait();
  const int D = p.dims[3], half = D / 2, cpr = half / 8;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t rem = i;
    const int c = int(rem % cpr); rem /= cpr;
    const int hg = int(rem % hgroups); rem /= hgroups;
    const int s = int(rem % p.dims[1]);
    const int b = int(rem / p.dims[1]);
    const int pos0 = p.pos ? p.pos[b * p.pos_stride] : 0;
    float cs[8], sn[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float fh, fl;
      rope_freq(p.freq, c * 8 + j, D, fh, fl);
      rope_sincos(s + pos0, fh, fl, sn[j], cs[j]);
    }
    const int h_end = min(p.dims[2], (hg + 1) * ROPE_HG);
    for (int h = hg * ROPE_HG; h < h_end; ++h) {
      const int64_t off = b * p.st[0] + s * p.st[1] + h * p.st[2] + c * 8;
      const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(p.x) + off;
      __nv_bfloat16* y = static_cast<__nv_bfloat16*>(p.y) + off;
      float a[8], bb[8], oa[8], ob[8];
      load16(x, a);
      load16(x + half, bb);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        oa[j] = a[j] * cs[j] - bb[j] * sn[j];
        ob[j] = bb[j] * cs[j] + a[j] * sn[j];
      }
      store16(y, oa);
      store16(y + half, ob);
    }
  }
}

cudaError_t launch_rope(const RopeParams& p, cudaStream_t st) {
  if (p.dtype == FLUID_BF16 && !p.interleaved && p.st[3] == 1 && (p.dims[3] / 2) % 8 == 0 && p.st[0] % 8 == 0 &&
      p.st[1] % 8 == 0 && p.st[2] % 8 == 0 && aligned16(p.x) && aligned16(p.y)) {
    const int hgroups = (p.dims[2] + ROPE_HG - 1) / ROPE_HG;
    const int64_t total = (int64_t)p.dims[0] * p.dims[1] * hgroups * (p.dims[3] / 16);
    const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 8);
    return launch_k(rope_vec_kernel, grid, 256, 0, st, p, total, hgroups);
  }
  const int64_t total = (int64_t)p.dims[0] * p.dims[1] * p.dims[2] * (p.dims[3] / 2);
  const int threads = 256;
  const unsigned grid = (unsigned)std::min<int64_t>((total + threads - 1) / threads, 148 * 32);
  return p.dtype == FLUID_BF16 ? launch_k(rope_kernel<__nv_bfloat16>, grid, threads, 0, st, p, total)
                               : launch_k(rope_kernel<float>, grid, threads, 0, st, p, total);
}

// ---- ELTWISE ---------------------------------------------------------------------------------------
template <int OP>
__device__ __forceinline__ float elt_apply(float a, float b) {
  if (OP == ELT_ADD) return a + b;
  if (OP == ELT_MUL) return a * b;
  if (OP == ELT_GELU_ERF) return gelu_erf_fast(a);
  if (OP == ELT_GELU_TANH) return gelu_tanh(a);
  if (OP == ELT_SILU) return silu(a);
  return silu(a) * b;
}

// One 16-byte chunk per thread per operand, two chunks in flight; WIDE (bf16 graphs, ADD only)
// lets operands / result be the fp32 copies of residual-stream tensors.
template <typename T, bool VECTOR, int OP, bool WIDE>
__global__ void __launch_bounds__(256) eltwise_kernel(EltParams p) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int V = VECTOR ? VecOf<T>::N : 1;
  constexpr bool BINARY = OP == ELT_ADD || OP == ELT_MUL || OP == ELT_SILU_MUL;
  T* y = static_cast<T*>(p.y);
  float* yf = static_cast<float*>(p.y);
  const bool a_f32 = WIDE && p.a_f32, b_f32 = WIDE && p.b_f32, y_wide = WIDE && p.y_f32;
  const int64_t nch = p.n / V;
  const int64_t c0 = ((int64_t)blockIdx.x * blockDim.x * 2) + threadIdx.x;
  float va[2][V], vb[2][V];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int64_t c = c0 + u * (int64_t)blockDim.x;
    if (c < nch) {
      norm_load<T, V>(p.a, a_f32, (size_t)c * V, 0, va[u]);
      if (BINARY) norm_load<T, V>(p.b, b_f32, (size_t)c * V, 0, vb[u]);
    }
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int64_t c = c0 + u * (int64_t)blockDim.x;
    if (c < nch) {
#pragma unroll
      for (int i = 0; i < V; ++i) va[u][i] = elt_apply<OP>(va[u][i], BINARY ? vb[u][i] : 0.f);
      if (VECTOR) {
        if (y_wide || sizeof(T) == 4) {
#pragma unroll
          for (int i = 0; i < V; i += 4)
            *reinterpret_cast<float4*>(yf + c * V + i) = make_float4(va[u][i], va[u][i + 1], va[u][i + 2], va[u][i + 3]);
        } else {
          float t8[VecOf<T>::N];
#pragma unroll
          for (int i = 0; i < V; ++i) t8[i] = va[u][i];
          store16(y + c * V, t8);
        }
      } else {
        if (y_wide) yf[c] = va[u][0];
        else y[c] = from_f<T>(va[u][0]);
      }
    }
  }
}

template <typename T, bool VECTOR>
static cudaError_t eltwise_v(const EltParams& p, unsigned grid, cudaStream_t st) {
  const bool wide = sizeof(T) == 2 && (p.a_f32 || p.b_f32 || p.y_f32);
  switch (p.op) {
    case ELT_ADD:
      return wide ? launch_k(eltwise_kernel<T, VECTOR, ELT_ADD, true>, grid, 256, 0, st, p)
                  : launch_k(eltwise_kernel<T, VECTOR, ELT_ADD, false>, grid, 256, 0, st, p);
    case ELT_MUL: return launch_k(eltwise_kernel<T, VECTOR, ELT_MUL, false>, grid, 256, 0, st, p);
    case ELT_GELU_ERF: return launch_k(eltwise_kernel<T, VECTOR, ELT_GELU_ERF, false>, grid, 256, 0, st, p);
    case ELT_GELU_TANH: return launch_k(eltwise_kernel<T, VECTOR, ELT_GELU_TANH, false>, grid, 256, 0, st, p);
    case ELT_SILU: return launch_k(eltwise_kernel<T, VECTOR, ELT_SILU, false>, grid, 256, 0, st, p);
    default: return launch_k(eltwise_kernel<T, VECTOR, ELT_SILU_MUL, false>, grid, 256, 0, st, p);
  }
}

template <typename T>
static cudaError_t eltwise_t(const EltParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.n % V == 0 && aligned16(p.a) && aligned16(p.y) && (!p.b || aligned16(p.b));
  const int64_t nch = p.n / (vec ? V : 1);
  const unsigned grid = (unsigned)((nch + 511) / 512);
  return vec ? eltwise_v<T, true>(p, grid, st) : eltwise_v<T, false>(p, grid, st);
}

cudaError_t launch_eltwise(const EltParams& p, cudaStream_t st) {
  return p.dtype == FLUID_BF16 ? eltwise_t<__nv_bfloat16>(p, st) : eltwise_t<float>(p, st);
}

// ---- PERMUTE ---------------------------------------------------------------------------------------
// Dims arrive sorted by output stride (slowest first), so a linear index over them walks the
// output contiguously.
struct PermSorted {
  int dims[5];
  int64_t xs[5], ys[5];
};

// Class A: the contiguous dim is the same on both sides -> move 16-byte (or element) rows.
template <typename E>
__global__ void permute_rows_kernel(const E* __restrict__ x, E* __restrict__ y, PermSorted s, int64_t total) {
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t rem = i, xo = 0, yo = 0;
#pragma unroll
    for (int k = 4; k >= 0; --k) {
      const int c = int(rem % s.dims[k]);
      rem /= s.dims[k];
      xo += c * s.xs[k];
      yo += c * s.ys[k];
    }
    y[yo] = x[xo];
  }
}

// The same for a dense output of fewer than 2^31 units (the usual case): the output offset of unit i is i
// itself, the input offset comes from 32-bit divisions, and a thread moves four units that are a quarter
// of the tensor apart (four loads in flight before the first store).
template <typename E>
__global__ void __launch_bounds__(256) permute_rows32_kernel(const E* __restrict__ x, E* __restrict__ y, PermSorted s, uint32_t total) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t quarter = (total + 3u) / 4u;
  const uint32_t d4 = uint32_t(s.dims[4]), d3 = uint32_t(s.dims[3]), d2 = uint32_t(s.dims[2]), d1 = uint32_t(s.dims[1]);
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < quarter; i += gridDim.x * blockDim.x) {
    E v[4];
    uint32_t idx[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      idx[u] = i + uint32_t(u) * quarter;
      if (idx[u] < total) {
        uint32_t rem = idx[u];
        const uint32_t c4 = rem % d4; rem /= d4;
        const uint32_t c3 = rem % d3; rem /= d3;
        const uint32_t c2 = rem % d2; rem /= d2;
        const uint32_t c1 = rem % d1; rem /= d1;
        const int64_t xo = (int64_t)c4 * s.xs[4] + (int64_t)c3 * s.xs[3] + (int64_t)c2 * s.xs[2] + (int64_t)c1 * s.xs[1] + (int64_t)rem * s.xs[0];
        v[u] = x[xo];
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (idx[u] < total) y[idx[u]] = v[u];
  }
}

// Class A where rows are short (<= 512 bytes) and the dim that follows them differs between input and output,
// e.g. [B,S,nh,D] -> [B,nh,S,D]: moving one row at a time touches DRAM in isolated 128-256-byte pieces on
// one side. Here a CTA moves a TP x TQ block of rows (16 x 8, or 8 x 8 for 512-byte rows) through shared memory: it reads TQ runs of TP rows that
// are contiguous in the input and writes TP runs of TQ rows that are contiguous in the output (2-4 KB each).
// Units are 16 bytes; U units per row; slot 3 of the sorted dims is the output-next dim Q, slot pk the
// input-next dim P; the other two dims are spread over the grid.
template <int U>
__global__ void __launch_bounds__(256) permute_rows_tile_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, PermSorted s, int pk,
                                                                int tiles_p, int tiles_q) {
  constexpr int TP = U == 32 ? 8 : 16, TQ = 8, N = TP * TQ * U, PER = N / 256;   // at most 32 KB of shared memory
  __shared__ uint4 tile[N];
  pdl_launch_dependents();
  int64_t blk = blockIdx.x;
  const int tq = int(blk % tiles_q); blk /= tiles_q;
  const int tp = int(blk % tiles_p); blk /= tiles_p;
  int64_t xo = 0, yo = 0;
#pragma unroll
  for (int k = 2; k >= 0; --k) {
    if (k == pk) continue;
    const int c = int(blk % s.dims[k]);
    blk /= s.dims[k];
    xo += c * s.xs[k];
    yo += c * s.ys[k];
  }
  const int p0 = tp * TP, q0 = tq * TQ, dp = s.dims[pk], dq = s.dims[3];
  const int64_t xp = s.xs[pk], xq = s.xs[3], yp = s.ys[pk], yq = s.ys[3];
  pdl_wait();
  uint4 v[PER];
#pragma unroll
  for (int j = 0; j < PER; ++j) {       // input order: u fastest, then p, then q
    const int e = threadIdx.x + 256 * j;
    const int u = e % U, pp = (e / U) % TP, qq = e / (U * TP);
    v[j] = make_uint4(0u, 0u, 0u, 0u);
    if (p0 + pp < dp && q0 + qq < dq) v[j] = x[xo + (p0 + pp) * xp + (q0 + qq) * xq + u];
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) tile[threadIdx.x + 256 * j] = v[j];   // [q][p][u]
  __syncthreads();
#pragma unroll
  for (int j = 0; j < PER; ++j) {       // output order: u fastest, then q, then p
    const int e = threadIdx.x + 256 * j;
    const int u = e % U, qq = (e / U) % TQ, pp = e / (U * TQ);
    if (p0 + pp < dp && q0 + qq < dq) y[yo + (p0 + pp) * yp + (q0 + qq) * yq + u] = tile[(qq * TP + pp) * U + u];
  }
}

// Class B: the contiguous dim changes -> shared-memory tile transpose. Tile = 64 (x-fast dim I)
// by 64 (y-fast dim O); the odd row pitch keeps both sweeps free of bank conflicts.
template <typename E>
__global__ void permute_tile_kernel(const E* __restrict__ x, E* __restrict__ y, PermSorted s, int di, int dn,
                                    int tiles_i, int tiles_o) {
  pdl_launch_dependents();
  pdl_wait();
  // s.dims[4] is the output-fast dim O (extent dn); s.dims[3] holds the input-fast dim I (extent di)
  __shared__ E tile[64][65];
  int64_t blk = blockIdx.x;
  const int ti = int(blk % tiles_i); blk /= tiles_i;
  const int to = int(blk % tiles_o); blk /= tiles_o;
  int64_t xo = 0, yo = 0;
#pragma unroll
  for (int k = 2; k >= 0; --k) {
    const int c = int(blk % s.dims[k]);
    blk /= s.dims[k];
    xo += c * s.xs[k];
    yo += c * s.ys[k];
  }
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;  // 256 threads: 64 x 4
  const int i0 = ti * 64, o0 = to * 64;
  // read: threads sweep I (contiguous in x)
  for (int r = ty; r < 64; r += 4) {
    const int o = o0 + r, i = i0 + tx;
    if (o < dn && i < di) tile[r][tx] = x[xo + (int64_t)o * s.xs[4] + (int64_t)i * s.xs[3]];
  }
  __syncthreads();
  // write: threads sweep O (contiguous in y)
  for (int r = ty; r < 64; r += 4) {
    const int i = i0 + r, o = o0 + tx;
    if (o < dn && i < di) y[yo + (int64_t)i * s.ys[3] + (int64_t)o * s.ys[4]] = tile[tx][r];
  }
}

// Class B for 16-bit elements with 16-byte accesses on both sides. Tile = 64 (O) x 64 (I). A thread
// reads 8 consecutive I (one 16-byte load) and parks them as four 32-bit words in a tile of 33-word
// rows (word w of row o holds I = 2w, 2w + 1): with the odd pitch both sweeps are free of bank
// conflicts. For the output a thread takes word w of 8 consecutive rows O, splits the halves and
// writes two 16-byte runs: 8 consecutive O of output row I = 2w and of row I = 2w + 1.
// Needs: both extents multiples of 8, every other stride a multiple of 8 elements, 16-byte aligned bases.
__global__ void __launch_bounds__(256) permute_tile16_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, PermSorted s,
                                                             int di, int dn, int tiles_i, int tiles_o) {
  pdl_launch_dependents();
  __shared__ uint32_t tile[64 * 33];
  int64_t blk = blockIdx.x;
  const int ti = int(blk % tiles_i); blk /= tiles_i;
  const int to = int(blk % tiles_o); blk /= tiles_o;
  int64_t xo = 0, yo = 0;
#pragma unroll
  for (int k = 2; k >= 0; --k) {
    const int c = int(blk % s.dims[k]);
    blk /= s.dims[k];
    xo += c * s.xs[k];
    yo += c * s.ys[k];
  }
  const int i0 = ti * 64, o0 = to * 64;
  pdl_wait();
  // read: lane = (row within a group of 4, 16-byte unit of the row); 8 lanes cover one 128-byte row segment
  {
    const int ig = threadIdx.x & 7, orow = threadIdx.x >> 3;   // 32 rows per pass
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int ol = orow + 32 * pass, o = o0 + ol, i = i0 + ig * 8;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (o < dn && i < di) v = *reinterpret_cast<const uint4*>(x + xo + (int64_t)o * s.xs[4] + i);
      uint32_t* dst = tile + ol * 33 + ig * 4;
      dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
  }
  __syncthreads();
  // write: lane = (group of 8 rows O: 4 per warp, word column w: 8 per warp)
  {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int og = (warp & 1) * 4 + (lane >> 3), w = (warp >> 1) * 8 + (lane & 7);   // og 0..7, w 0..31
    uint32_t q[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) q[e] = tile[(og * 8 + e) * 33 + w];
    const int i = i0 + 2 * w, o = o0 + og * 8;
    if (o < dn && i < di) {
      uint4 lo, hi;   // low halves = row I = 2w, high halves = row I = 2w + 1
      lo.x = __byte_perm(q[0], q[1], 0x5410); hi.x = __byte_perm(q[0], q[1], 0x7632);
      lo.y = __byte_perm(q[2], q[3], 0x5410); hi.y = __byte_perm(q[2], q[3], 0x7632);
      lo.z = __byte_perm(q[4], q[5], 0x5410); hi.z = __byte_perm(q[4], q[5], 0x7632);
      lo.w = __byte_perm(q[6], q[7], 0x5410); hi.w = __byte_perm(q[6], q[7], 0x7632);
      uint16_t* dst = y + yo + (int64_t)i * s.ys[3] + o;
      *reinterpret_cast<uint4*>(dst) = lo;
      *reinterpret_cast<uint4*>(dst + s.ys[3]) = hi;
    }
  }
}

template <typename E>
static void permute_dispatch(const PermuteParams& p, cudaStream_t st) {
  // order dims by output stride, slowest first; pad to 5 with unit dims in front
  int idx[5], n = 0;
  for (int j = 0; j < p.rank; ++j)
    if (p.dims[j] > 1) idx[n++] = j;
  std::sort(idx, idx + n, [&](int a, int b) { return p.ys[a] > p.ys[b]; });
  PermSorted s;
  for (int k = 0; k < 5; ++k) { s.dims[k] = 1; s.xs[k] = 0; s.ys[k] = 0; }
  for (int k = 0; k < n; ++k) {
    const int j = idx[k], dst = 5 - n + k;
    s.dims[dst] = p.dims[j]; s.xs[dst] = p.xs[j]; s.ys[dst] = p.ys[j];
  }
  const E* x = static_cast<const E*>(p.x) + p.x_offset;
  E* y = static_cast<E*>(p.y);
  int64_t total = 1;
  for (int k = 0; k < 5; ++k) total *= s.dims[k];
  const bool same_inner = n == 0 || s.xs[4] == 1;
  if (same_inner) {
    // widen to 16-byte units when the shared fast dim and every other stride allow it
    constexpr int W = 16 / sizeof(E);
    bool wide = n > 0 && s.dims[4] % W == 0 && aligned16(x) && aligned16(y);
    for (int k = 0; k < 4 && wide; ++k)
      if (s.dims[k] > 1 && (s.xs[k] % W || s.ys[k] % W)) wide = false;
    if (wide) {
      PermSorted w = s;
      w.dims[4] /= W;
      for (int k = 0; k < 4; ++k) { w.xs[k] /= W; w.ys[k] /= W; }
      const int64_t tw = total / W;
      // dense output in sorted-stride order: unit i of y is at offset i
      bool dense = w.ys[4] == 1 && tw < (int64_t(1) << 31);
      for (int k = 3; k >= 0 && dense; --k)
        if (w.dims[k] > 1) dense = w.ys[k] == w.ys[k + 1] * w.dims[k + 1];   // (unit dims pad the front)
      // short rows whose next dim differs between input and output: block-of-rows kernel
      if (dense && (w.dims[4] == 8 || w.dims[4] == 16 || w.dims[4] == 32) && w.dims[3] > 1 && w.xs[3] != w.dims[4]) {
        int pk = -1;
        for (int k = 0; k < 3; ++k)
          if (w.dims[k] > 1 && w.xs[k] == w.dims[4]) pk = k;
        if (pk >= 0) {
          const int tp_rows = w.dims[4] == 32 ? 8 : 16;
          const int tiles_p = (w.dims[pk] + tp_rows - 1) / tp_rows, tiles_q = (w.dims[3] + 7) / 8;
          int64_t blocks = (int64_t)tiles_p * tiles_q;
          for (int k = 0; k < 3; ++k)
            if (k != pk) blocks *= w.dims[k];
          if (blocks < (int64_t(1) << 31)) {
            const uint4* xv = reinterpret_cast<const uint4*>(x);
            uint4* yv = reinterpret_cast<uint4*>(y);
            if (w.dims[4] == 8) launch_k(permute_rows_tile_kernel<8>, (unsigned)blocks, 256, 0, st, xv, yv, w, pk, tiles_p, tiles_q);
            else if (w.dims[4] == 16) launch_k(permute_rows_tile_kernel<16>, (unsigned)blocks, 256, 0, st, xv, yv, w, pk, tiles_p, tiles_q);
            else launch_k(permute_rows_tile_kernel<32>, (unsigned)blocks, 256, 0, st, xv, yv, w, pk, tiles_p, tiles_q);
            return;
          }
        }
      }
      if (dense) {
        const unsigned grid32 = (unsigned)std::min<int64_t>((tw / 4 + 255) / 256, 148 * 16);
        launch_k(permute_rows32_kernel<uint4>, std::max(1u, grid32), 256, 0, st, reinterpret_cast<const uint4*>(x), reinterpret_cast<uint4*>(y),
                 w, (uint32_t)tw);
        return;
      }
      const unsigned grid = (unsigned)std::min<int64_t>((tw + 255) / 256, 148 * 16);
      launch_k(permute_rows_kernel<uint4>, grid, 256, 0, st, reinterpret_cast<const uint4*>(x), reinterpret_cast<uint4*>(y), w, tw);
    } else {
      const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 16);
      launch_k(permute_rows_kernel<E>, grid, 256, 0, st, x, y, s, total);
    }
    return;
  }
  // find the input-fast dim and move it to slot 3
  int xi = -1;
  for (int k = 0; k < 4; ++k)
    if (s.dims[k] > 1 && s.xs[k] == 1) xi = k;
  if (xi < 0) {
    const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 16);
    launch_k(permute_rows_kernel<E>, grid, 256, 0, st, x, y, s, total);
    return;
  }
  PermSorted t = s;
  // rotate slot xi to position 3, keeping the others in order
  int dI = s.dims[xi]; int64_t xI = s.xs[xi], yI = s.ys[xi];
  for (int k = xi; k < 3; ++k) { t.dims[k] = s.dims[k + 1]; t.xs[k] = s.xs[k + 1]; t.ys[k] = s.ys[k + 1]; }
  t.dims[3] = dI; t.xs[3] = xI; t.ys[3] = yI;
  const int tiles_i = (t.dims[3] + 63) / 64, tiles_o = (t.dims[4] + 63) / 64;
  const int64_t blocks = (int64_t)tiles_i * tiles_o * t.dims[0] * t.dims[1] * t.dims[2];
  if (sizeof(E) == 2) {
    bool wide = t.dims[3] % 8 == 0 && t.dims[4] % 8 == 0 && t.xs[3] == 1 && t.ys[4] == 1 && t.xs[4] % 8 == 0 && t.ys[3] % 8 == 0 &&
                aligned16(x) && aligned16(y);
    for (int k = 0; k < 3 && wide; ++k)
      if (t.dims[k] > 1 && (t.xs[k] % 8 || t.ys[k] % 8)) wide = false;
    if (wide) {
      launch_k(permute_tile16_kernel, (unsigned)blocks, 256, 0, st, reinterpret_cast<const uint16_t*>(x), reinterpret_cast<uint16_t*>(y), t,
               t.dims[3], t.dims[4], tiles_i, tiles_o);
      return;
    }
  }
  launch_k(permute_tile_kernel<E>, (unsigned)blocks, 256, 0, st, x, y, t, t.dims[3], t.dims[4], tiles_i, tiles_o);
}

// FLUID_PERMUTE_TMA=0 in the environment keeps every transform on the register kernels (A/B timing).
static bool permute_tma_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("FLUID_PERMUTE_TMA");
    return !(e && e[0] == '0');
  }();
  return on;
}

cudaError_t launch_permute(const PermuteParams& p, cudaStream_t st) {
  if (permute_tma_enabled()) {
    cudaError_t err = cudaSuccess;
    if (launch_permute_tma(p, p.status, st, &err)) return err;
  }
  if (p.esize == 2) permute_dispatch<uint16_t>(p, st);
  else permute_dispatch<uint32_t>(p, st);
  return cudaGetLastError();
}

}  // namespace fluid
