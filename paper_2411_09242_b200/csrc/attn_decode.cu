// Attention of one decoding step against a key/value cache (single new token per sequence).
//
// The step is bound by reading the cache once: per (sequence, head) t+1 rows of D keys and D values, one
// multiply-add per byte pair. No tensor cores: rows stream through the SM in 16-byte pieces.
//
// Work split: one thread-block cluster of up to 8 CTAs per (sequence, query head); CTA r of the cluster takes a
// contiguous share of the rows 0..t. Inside a CTA a row is owned by LPR = D / (16 bytes of elements)
// adjacent lanes (a warp covers 32 / LPR rows per load instruction); every such lane group keeps a running
// (max, sum, output) triple in the base-2 online-softmax form; its rows of keys and values arrive through a
// per-lane ring of asynchronous copies in shared memory, several rows deep. Triples are merged lane group -> warp
// (shuffles) -> CTA (shared memory) -> cluster (each CTA stores its triple into CTA 0's shared memory; one cluster
// barrier), and CTA 0 writes the D outputs.
// The row of the new token comes from the step's own k and v operands, and the CTA that meets it stores it
// as row t of the caches: no row is read from the cache in the launch that writes it.
//
// Nothing here spins: the only waits are __syncthreads and the hardware cluster barrier.
#include <algorithm>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

constexpr int kSplits = 8;    // most CTAs per cluster = row ranges per (sequence, head); a launch uses 1 to 8
constexpr int kWarps = 8;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <typename T>
__device__ __forceinline__ void unpack16(const uint4& q, float (&v)[VecOf<T>::N]);
template <>
__device__ __forceinline__ void unpack16<float>(const uint4& q, float (&v)[4]) {
  v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y); v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
}
template <>
__device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& q, float (&v)[8]) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

constexpr int kStages = 8;    // ring depth: rows of K and of V a lane group has in flight, plus the one being consumed

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

// weight of a partial with maximum m inside a merge whose maximum is M (an empty partial has m = -inf)
__device__ __forceinline__ float merge_weight(float m, float M) { return m == -INFINITY ? 0.f : exp2f(m - M); }

template <typename T>
__device__ __forceinline__ uint4 pack16(const float (&v)[VecOf<T>::N]);
template <>
__device__ __forceinline__ uint4 pack16<float>(const float (&v)[4]) {
  return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
}
template <>
__device__ __forceinline__ uint4 pack16<__nv_bfloat16>(const float (&v)[8]) {
  return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
}

// Rotary embedding (pairs (d, d + D/2)) of one row of D = LPR * V elements spread over LPR adjacent lanes, lane li
// holding elements li*V .. li*V + V-1, at position pos. Every lane of the warp must call it.
template <int V, int LPR>
__device__ __forceinline__ void rotate_row(float (&x)[V], int li, int pos, const RopeFreq& freq) {
  constexpr int D = LPR * V, half = D / 2;
  float partner[V];
#pragma unroll
  for (int i = 0; i < V; ++i) partner[i] = LPR > 1 ? __shfl_xor_sync(0xffffffffu, x[i], LPR / 2) : x[(i + V / 2) % V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int d = li * V + i;
    const int dd = d < half ? d : d - half;
    float sn, cs;
    float fh, fl;
    rope_freq(freq, dd, D, fh, fl);
    rope_sincos(pos, fh, fl, sn, cs);
    x[i] = d < half ? x[i] * cs - partner[i] * sn : x[i] * cs + partner[i] * sn;
  }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kWarps * 32) attn_decode_kernel(AttnDecodeParams p) {
  constexpr int V = VecOf<T>::N;
  constexpr int D = LPR * V;
  constexpr int GPW = 32 / LPR;          // rows per warp and load instruction
  constexpr int RPI = GPW * kWarps;      // rows per CTA and load instruction
  __shared__ float part[kWarps][D + 2];  // per warp: D outputs, max, sum
  __shared__ float cl[kSplits][D + 2];   // per CTA of the cluster (filled in CTA 0 only)
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane / LPR, li = lane % LPR;
  const int split = blockIdx.x, n_split = gridDim.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.NH / p.NKV);
  const int t = p.pos[b * p.pos_stride];   // a graph input: nothing in this run writes it
  const bool t_ok = t >= 0 && t < p.Tmax;
  const int n = t_ok ? t + 1 : 0;
  const int chunk = ((n + n_split - 1) / n_split + RPI - 1) / RPI * RPI;
  const int r0 = split * chunk, r1 = min(n, r0 + chunk);
  const int r1c = min(r1, t);   // rows before t come from the caches
  const int64_t row_stride = (int64_t)p.NKV * D;
  T* kc = static_cast<T*>(p.kc) + ((int64_t)b * p.Tmax * p.NKV + g) * D + li * V;
  T* vc = static_cast<T*>(p.vc) + ((int64_t)b * p.Tmax * p.NKV + g) * D + li * V;
  // Each lane copies the 16 bytes of K and of V it will consume itself into a private ring in shared memory
  // (asynchronous copies, kStages deep): it only ever reads back its own copies, so the ring needs no barrier, and the
  // bytes in flight are set by the ring's depth. The cache rows were written by earlier runs, not by this run's
  // earlier steps: the first copies are requested before the wait for the previous step.
  extern __shared__ __align__(16) unsigned char ring_raw[];
  const uint32_t my_ring = static_cast<uint32_t>(__cvta_generic_to_shared(ring_raw)) + uint32_t(warp) * (kStages * 2 * 32 * 16) + uint32_t(lane) * 16;
  auto slot = [&](int i, int which) { return my_ring + uint32_t(i % kStages) * (2 * 32 * 16) + uint32_t(which) * (32 * 16); };
  const int jbase = r0 + warp * GPW + grp;
  const int n_slots = r0 + warp * GPW < r1c ? (r1c - (r0 + warp * GPW) + RPI - 1) / RPI : 0;
  auto fill = [&](int i) {
    const int j = jbase + i * RPI;
    const bool ok = i < n_slots && j < r1c;
    const int64_t off = ok ? j * row_stride : 0;   // a zero-filled copy reads nothing, its address stays inside the cache
    cp_async16(slot(i, 0), kc + off, ok);
    cp_async16(slot(i, 1), vc + off, ok);
  };
  for (int i = 0; i < kStages - 1; ++i) {
    fill(i);
    cp_async_commit();
  }
  pdl_wait();
  if (!t_ok) {   // the same in every CTA of the cluster (one sequence, one head): nobody reaches the cluster barrier
    cp_async_wait<0>();
    if (threadIdx.x == 0 && split == 0 && h == 0) atomicOr(p.status, 0x10u);
    return;
  }

  float qv[V];
  {
    const uint4 raw = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.q) + b * p.q_sb + h * p.q_sh + li * V);
    unpack16<T>(raw, qv);
    if (p.rope) rotate_row<V, LPR>(qv, li, t, p.rope_freq);
#pragma unroll
    for (int i = 0; i < V; ++i) qv[i] *= p.scale_log2;
  }
  // the new token's key (rotated here when the step carries the rotary embedding) and value
  uint4 k_fresh = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.k) + b * p.k_sb + g * p.k_sh + li * V);
  const uint4 v_fresh = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.v) + b * p.v_sb + g * p.v_sh + li * V);
  if (p.rope) {
    float kf[V];
    unpack16<T>(k_fresh, kf);
    rotate_row<V, LPR>(kf, li, t, p.rope_freq);
    k_fresh = pack16<T>(kf);   // rounded as the cache will hold it: later steps read exactly what this one used
  }

  float m = -INFINITY, l = 0.f, o[V];
#pragma unroll
  for (int i = 0; i < V; ++i) o[i] = 0.f;

  // rows before t come from the caches, through the ring. The loop bound is the warp's, not the lane group's: every
  // lane takes part in the shuffles of every pass; a group whose row is past the end contributes nothing
#pragma unroll 1
  for (int i = 0; i < n_slots; ++i) {
    cp_async_wait<kStages - 2>();   // this lane's copies of slot i have landed
    const uint4 kq = lds128(slot(i, 0)), vq = lds128(slot(i, 1));
    fill(i + kStages - 1);          // refills the slot read one pass ago
    cp_async_commit();
    const bool live = jbase + i * RPI < r1c;
    float kf[V], vf[V];
    unpack16<T>(kq, kf);
    unpack16<T>(vq, vf);
    float sc = 0.f;
#pragma unroll
    for (int e = 0; e < V; ++e) sc = fmaf(qv[e], kf[e], sc);
    // the lanes of a group hold partial dot products of the same row; the exchange stays inside the group (LPR is a
    // power of two, groups are aligned)
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, off);
    if (live) {
      const float m_new = fmaxf(m, sc);
      const float corr = merge_weight(m, m_new), e = exp2f(sc - m_new);
      l = fmaf(l, corr, e);
#pragma unroll
      for (int d = 0; d < V; ++d) o[d] = fmaf(e, vf[d], o[d] * corr);
      m = m_new;
    }
  }
  cp_async_wait<0>();
  // row t, the new token: from the step's own operands, in the first warp of the CTA whose range holds it; that
  // warp's first lane group counts it and stores it as row t of the caches
  if (t >= r0 && t < r1 && warp == 0) {
    float kf[V], vf[V];
    unpack16<T>(k_fresh, kf);
    unpack16<T>(v_fresh, vf);
    float sc = 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) sc = fmaf(qv[i], kf[i], sc);
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, off);
    if (grp == 0) {
      const float m_new = fmaxf(m, sc);
      const float corr = merge_weight(m, m_new), e = exp2f(sc - m_new);
      l = l * corr + e;
#pragma unroll
      for (int i = 0; i < V; ++i) o[i] = fmaf(e, vf[i], o[i] * corr);
      m = m_new;
      *reinterpret_cast<uint4*>(kc + t * row_stride) = k_fresh;
      *reinterpret_cast<uint4*>(vc + t * row_stride) = v_fresh;
    }
  }

  // lane groups of a warp -> one triple per warp
#pragma unroll
  for (int off = LPR; off < 32; off <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    const float l2 = __shfl_xor_sync(0xffffffffu, l, off);
    const float M = fmaxf(m, m2);
    const float a = merge_weight(m, M), a2 = merge_weight(m2, M);
    l = l * a + l2 * a2;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const float o2 = __shfl_xor_sync(0xffffffffu, o[i], off);
      o[i] = o[i] * a + o2 * a2;
    }
    m = M;
  }
  if (grp == 0) {
#pragma unroll
    for (int i = 0; i < V; ++i) part[warp][li * V + i] = o[i];
    if (li == 0) {
      part[warp][D] = m;
      part[warp][D + 1] = l;
    }
  }
  __syncthreads();
  // warps -> one triple per CTA, stored into CTA 0's table
  if (threadIdx.x < D + 2) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, part[w][D]);
    float val;
    if (threadIdx.x == D) {
      val = M;
    } else {
      const int col = threadIdx.x < D ? threadIdx.x : D + 1;
      val = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) val = fmaf(merge_weight(part[w][D], M), part[w][col], val);
    }
    st_cluster_f32(map_to_cta(smem_addr(&cl[split][threadIdx.x]), 0u), val);
  }
  cluster_sync_all();
  if (split != 0) return;
  if (threadIdx.x < D) {
    float M = -INFINITY;
#pragma unroll
    for (int r = 0; r < n_split; ++r) M = fmaxf(M, cl[r][D]);
    float acc = 0.f, L = 0.f;
    for (int r = 0; r < n_split; ++r) {
      const float a = merge_weight(cl[r][D], M);
      acc = fmaf(a, cl[r][threadIdx.x], acc);
      L = fmaf(a, cl[r][D + 1], L);
    }
    static_cast<T*>(p.out)[b * p.o_sb + h * p.o_sh + threadIdx.x] = from_f<T>(acc / L);
  }
}

template <typename T, int LPR>
cudaError_t launch_one(const AttnDecodeParams& p, cudaStream_t st) {
  constexpr size_t smem = size_t(kWarps) * kStages * 2 * 32 * 16;
  static const cudaError_t attr_rc = cudaFuncSetAttribute(attn_decode_kernel<T, LPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (attr_rc != cudaSuccess) return attr_rc;
  // row ranges per (sequence, head): as many as still leave the whole launch resident at once (three CTAs fit an SM);
  // a second, partial wave would run with few bytes in flight
  const int64_t heads = (int64_t)p.B * p.NH;
  const int splits = (int)std::max<int64_t>(1, std::min<int64_t>(kSplits, (148 * 3) / heads));
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)splits, (unsigned)p.NH, (unsigned)p.B);
  cfg.blockDim = dim3(kWarps * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, attn_decode_kernel<T, LPR>, p);
}

template <typename T>
cudaError_t launch_t(const AttnDecodeParams& p, cudaStream_t st) {
  switch (p.D / VecOf<T>::N) {
    case 1: return launch_one<T, 1>(p, st);
    case 2: return launch_one<T, 2>(p, st);
    case 4: return launch_one<T, 4>(p, st);
    case 8: return launch_one<T, 8>(p, st);
    case 16: return launch_one<T, 16>(p, st);
    case 32:
      if constexpr (sizeof(T) == 4) return launch_one<T, 32>(p, st);
      break;
  }
  return cudaErrorInvalidValue;
}

inline bool al16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

}  // namespace

bool attn_decode_supported(int dtype, int D) {
  if (dtype != FLUID_BF16 && dtype != FLUID_F32) return false;
  const int v = dtype == FLUID_BF16 ? 8 : 4;
  if (D % v) return false;
  const int lpr = D / v;
  return D <= 128 && lpr >= 1 && lpr <= 32 && (lpr & (lpr - 1)) == 0;   // the merge steps use one thread per output column
}

cudaError_t launch_attn_decode(const AttnDecodeParams& p, cudaStream_t st) {
  if (!attn_decode_supported(p.dtype, p.D) || p.NKV < 1 || p.NH % p.NKV || p.B < 1 || p.B > 65535 || p.NH > 65535)
    return cudaErrorInvalidValue;
  const int v = p.dtype == FLUID_BF16 ? 8 : 4;
  const int64_t strides[8] = {p.q_sb, p.q_sh, p.k_sb, p.k_sh, p.v_sb, p.v_sh, p.o_sb, p.o_sh};
  for (int i = 0; i < 6; ++i)
    if (strides[i] % v) return cudaErrorInvalidValue;
  if (!al16(p.q) || !al16(p.k) || !al16(p.v) || !al16(p.kc) || !al16(p.vc)) return cudaErrorInvalidValue;
  return p.dtype == FLUID_BF16 ? launch_t<__nv_bfloat16>(p, st) : launch_t<float>(p, st);
}

}  // namespace fluid
