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
  const T* pos = p.pos ? static_cast<const T*>(p.pos) + (size_t)(t % p.S) * p.H : nullptr;
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

template <typename T>
static cudaError_t norm_t(const NormParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.width % V == 0 && aligned16(p.x) && (!p.y_lo || aligned16(p.y_lo)) && (!p.y_hi || aligned16(p.y_hi)) &&
                   aligned16(p.gamma) && (!p.beta || aligned16(p.beta)) && (!p.res || aligned16(p.res));
  const int nch = p.width / (vec ? V : 1);
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
    const float inv_freq = exp2f(-2.f * pr / p.dims[3] * log2f(p.base));
    float sn, cs;
    sincosf(idx[1] * inv_freq, &sn, &cs);
    const T* x = static_cast<const T*>(p.x);
    T* y = static_cast<T*>(p.y);
    const float a = to_f(x[base + d0 * p.st[3]]), b = to_f(x[base + d1 * p.st[3]]);
    y[base + d0 * p.st[3]] = from_f<T>(a * cs - b * sn);
    y[base + d1 * p.st[3]] = from_f<T>(b * cs + a * sn);
  }
}

cudaError_t launch_rope(const RopeParams& p, cudaStream_t st) {
  const int64_t total = (int64_t)p.dims[0] * p.dims[1] * p.dims[2] * (p.dims[3] / 2);
  const int threads = 256;
  const unsigned grid = (unsigned)std::min<int64_t>((total + threads - 1) / threads, 148 * 32);
  return p.dtype == FLUID_BF16 ? launch_k(rope_kernel<__nv_bfloat16>, grid, threads, 0, st, p, total)
                               : launch_k(rope_kernel<float>, grid, threads, 0, st, p, total);
}

// ---- ELTWISE ---------------------------------------------------------------------------------------
__device__ __forceinline__ float elt_apply(int op, float a, float b) {
  switch (op) {
    case ELT_ADD: return a + b;
    case ELT_MUL: return a * b;
    case ELT_GELU_ERF: return gelu_erf(a);
    case ELT_GELU_TANH: return gelu_tanh(a);
    case ELT_SILU: return silu(a);
    default: return silu(a) * b;
  }
}

template <typename T, bool VECTOR>
__global__ void eltwise_kernel(EltParams p) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int V = VECTOR ? VecOf<T>::N : 1;
  T* y = static_cast<T*>(p.y);
  float* yf = static_cast<float*>(p.y);
  const bool y_wide = p.y_f32 && sizeof(T) == 2;
  const int64_t nch = p.n / V;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < nch; c += (int64_t)gridDim.x * blockDim.x) {
    float va[V], vb[V];
    norm_load<T, V>(p.a, p.a_f32, (size_t)c * V, 0, va);
    if (p.b) norm_load<T, V>(p.b, p.b_f32, (size_t)c * V, 0, vb);
#pragma unroll
    for (int i = 0; i < V; ++i) va[i] = elt_apply(p.op, va[i], p.b ? vb[i] : 0.f);
    if (VECTOR) {
      if (y_wide || sizeof(T) == 4) {
#pragma unroll
        for (int i = 0; i < V; i += 4)
          *reinterpret_cast<float4*>(yf + c * V + i) = make_float4(va[i], va[i + 1], va[i + 2], va[i + 3]);
      } else {
        float t8[VecOf<T>::N];
#pragma unroll
        for (int i = 0; i < V; ++i) t8[i] = va[i];
        store16(y + c * V, t8);
      }
    } else {
      if (y_wide) yf[c] = va[0];
      else y[c] = from_f<T>(va[0]);
    }
  }
}

template <typename T>
static cudaError_t eltwise_t(const EltParams& p, cudaStream_t st) {
  constexpr int V = VecOf<T>::N;
  const bool vec = p.n % V == 0 && aligned16(p.a) && aligned16(p.y) && (!p.b || aligned16(p.b));
  const int64_t nch = p.n / (vec ? V : 1);
  const unsigned grid = (unsigned)std::min<int64_t>((nch + 255) / 256, 148 * 16);
  return vec ? launch_k(eltwise_kernel<T, true>, grid, 256, 0, st, p) : launch_k(eltwise_kernel<T, false>, grid, 256, 0, st, p);
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
  launch_k(permute_tile_kernel<E>, (unsigned)blocks, 256, 0, st, x, y, t, t.dims[3], t.dims[4], tiles_i, tiles_o);
}

cudaError_t launch_permute(const PermuteParams& p, cudaStream_t st) {
  if (p.esize == 2) permute_dispatch<uint16_t>(p, st);
  else permute_dispatch<uint32_t>(p, st);
  return cudaGetLastError();
}

}  // namespace fluid
