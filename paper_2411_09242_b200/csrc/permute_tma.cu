// Layout transforms as pure TMA traffic. Every warp of a CTA is an independent worker with its own ring of
// shared-memory boxes: a tiled bulk-tensor load fills a box, a tiled bulk-tensor store drains it, and the worker keeps
// `stages - 1` loads and one store in flight. Two shapes of transform qualify:
//
//  rows  (class A: [B,S,nh,D] -> [B,nh,S,D] and the like) - both sides share the fastest dim. Both tensor maps are
//        written in the OUTPUT's dim order (the input map with the input's strides), so one coordinate tuple addresses
//        a box on both sides, and the box is "R rows of the next-fastest output dim": the store is one dense run of R
//        rows, the load a gather of R row segments. No register ever holds the data; one lane per worker runs.
//
//  tiles (class B: [B,S,nh,D] -> [B,nh,D,S] and the like, 16-bit elements) - the input's fastest dim I and the
//        output's fastest dim O differ. A box is 64 (O) x 64 (I) elements, brought in with the 128-byte swizzle; the
//        warp transposes it IN PLACE (sixteen ldmatrix.x4.trans take the 64 8x8 blocks into registers, sixteen
//        stmatrix.x4 put block (o, i) back at (i, o), again in the swizzled order, so neither sweep has a bank
//        conflict) and the same box leaves as 64 rows of 64 O by a swizzled store.
//
// Ragged extents need no code: a load past the end fills zeros, a store past the end is clipped.
// Every wait is bounded; an expired one sets bit 0x400 of the status word and the worker drains and leaves.
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

constexpr int kMaxWarps = 8;
constexpr long long kWaitCycles = 3000000000LL;

struct PermTma {
  int n_box[5];          // boxes along each dim of the load's coordinate (fastest first)
  int box[5];            // box extent along each dim
  int total;             // boxes in all
  int stages;            // boxes in one worker's ring
  uint32_t stage_bytes;  // bytes of shared memory per box
  uint32_t box_bytes;    // bytes one full box brings in
  uint32_t* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void stsm_x4(uint32_t addr, const uint32_t* r) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};"
               ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

// kTranspose: the box is a swizzled 64 x 64 tile of 16-bit elements, transposed in place by the whole warp, and the
// store's first two coordinates are the load's swapped. Otherwise lane 0 alone moves boxes as they are.
template <bool kTranspose>
__global__ void __launch_bounds__(kMaxWarps * 32)
permute_tma_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_out,
                   const __grid_constant__ PermTma p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const uint32_t ring = ((raw + 1023u) & ~1023u) + uint32_t(warp * p.stages) * p.stage_bytes;
  const uint32_t bars = ((raw + 1023u) & ~1023u) + uint32_t(n_warps * p.stages) * p.stage_bytes + uint32_t(warp * p.stages) * 8u;
  pdl_launch_dependents();
  if (!kTranspose && lane != 0) return;
  if (lane == 0) {
    for (int s = 0; s < p.stages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8u * s), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_in)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_out)) : "memory");
  }
  if (kTranspose) __syncwarp();
  const int first = blockIdx.x * n_warps + warp, step = gridDim.x * n_warps;
  const int mine = first < p.total ? (p.total - first + step - 1) / step : 0;
  auto coords = [&](int k, int* c) {
    int item = first + k * step;
#pragma unroll
    for (int d = 0; d < 5; ++d) {
      c[d] = (item % p.n_box[d]) * p.box[d];
      item /= p.n_box[d];
    }
  };
  auto load = [&](int k) {
    int c[5];
    coords(k, c);
    const int s = k % p.stages;
    const uint32_t bar = bars + 8u * s, dst = ring + uint32_t(s) * p.stage_bytes;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(p.box_bytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&map_in)), "r"(bar), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4])
        : "memory");
  };
  pdl_wait();   // the input comes from the previous step; the output may still be read by it
  int issued = 0;   // loads issued (lane 0's count)
  if (lane == 0)
    for (; issued < mine && issued < p.stages; ++issued) load(issued);
  bool ok = true;
  int landed = 0;   // boxes whose load has been waited for
  for (int k = 0; k < mine; ++k) {
    const int s = k % p.stages;
    ok = mbar_wait(bars + 8u * s, uint32_t(k / p.stages) & 1u);
    if (kTranspose) ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    landed = k + 1;
    const uint32_t box = ring + uint32_t(s) * p.stage_bytes;
    if (kTranspose) {
      // lane -> (matrix m = lane / 8 of an x4 group, row r = lane % 8); block b = 4 j + m sits at block row b / 8,
      // block column b % 8; row r of block (R, C) starts at (8 R + r) * 128 + ((C ^ r) * 16) under the 128-byte swizzle
      const int m = lane >> 3, r = lane & 7;
      uint32_t q[16][4];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int b = 4 * j + m, R = b >> 3, C = b & 7;
        ldsm_x4_trans(box + uint32_t((8 * R + r) * 128 + ((C ^ r) << 4)), q[j]);
      }
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int b = 4 * j + m, R = b >> 3, C = b & 7;
        stsm_x4(box + uint32_t((8 * C + r) * 128 + ((R ^ r) << 4)), q[j]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
    }
    if (lane == 0) {
      int c[5];
      coords(k, c);
      if (kTranspose) { const int t = c[0]; c[0] = c[1]; c[1] = t; }
      asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
                   ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(box), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4])
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      // the store of box k - 1 has read its shared memory: that box takes the next load
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      if (k >= 1 && issued < mine) load(issued++);
    }
  }
  if (!ok && lane == 0) {
    if (p.status) atomicOr(p.status, 0x400u);
    // loads already issued must land before the shared memory goes (each wait bounded)
    for (int k = landed; k < issued; ++k) mbar_wait(bars + 8u * (k % p.stages), uint32_t(k / p.stages) & 1u);
  }
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // every store complete before the CTA exits
}

// Launch shape of the two forms: warps (workers) per CTA, boxes per worker, CTAs per SM, bytes per box (rows form).
// The defaults are the measured optimum on 0.5 GB transforms: about 100-130 KB of boxes per SM. Both deeper rings and
// more workers ran slower (rows: 6 boxes of 16 KB 6.4 TB/s, 8 boxes 5.8; tiles: 16 boxes of 8 KB 6.0 TB/s, 24 boxes 5.7),
// shallower ones starve (4 boxes of 16 KB 4.9 TB/s).
// FLUID_PERMUTE_TMA_CFG="wA,sA,cA,kbA,wB,sB,cB" in the environment overrides the defaults (for timing runs).
struct TmaCfg {
  int warps_a = 2, stages_a = 3, ctas_a = 1, box_kb_a = 16;
  int warps_b = 8, stages_b = 2, ctas_b = 1;
};

const TmaCfg& tma_cfg() {
  static const TmaCfg cfg = [] {
    TmaCfg c;
    if (const char* e = std::getenv("FLUID_PERMUTE_TMA_CFG")) {
      int v[7];
      if (std::sscanf(e, "%d,%d,%d,%d,%d,%d,%d", v, v + 1, v + 2, v + 3, v + 4, v + 5, v + 6) == 7) {
        auto clamp = [](int x, int lo, int hi) { return std::min(std::max(x, lo), hi); };
        c.warps_a = clamp(v[0], 1, kMaxWarps); c.stages_a = clamp(v[1], 2, 16); c.ctas_a = clamp(v[2], 1, 8);
        c.box_kb_a = clamp(v[3], 1, 32);
        c.warps_b = clamp(v[4], 1, kMaxWarps); c.stages_b = clamp(v[5], 2, 16); c.ctas_b = clamp(v[6], 1, 8);
      }
    }
    return c;
  }();
  return cfg;
}

template <bool kTranspose>
cudaError_t launch_form(const TensorMapStorage& m_in, const TensorMapStorage& m_out, PermTma q, int warps, int ctas_per_sm,
                        cudaStream_t st) {
  size_t smem = size_t(warps) * q.stages * (q.stage_bytes + 8) + 1024;
  // keep the ring inside what one SM can give `ctas_per_sm` CTAs
  while (smem * ctas_per_sm > 220 * 1024 && q.stages > 2) {
    --q.stages;
    smem = size_t(warps) * q.stages * (q.stage_bytes + 8) + 1024;
  }
  static size_t attr_bytes = 0;
  if (smem > attr_bytes) {
    cudaError_t e = cudaFuncSetAttribute(permute_tma_kernel<kTranspose>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_bytes = smem;
  }
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = (int64_t(q.total) + warps - 1) / warps;
  const unsigned grid = (unsigned)std::min<int64_t>(want, int64_t(sms) * ctas_per_sm);
  return launch_k(permute_tma_kernel<kTranspose>, grid, (unsigned)warps * 32, smem, st, *reinterpret_cast<const CUtensorMap*>(&m_in),
                  *reinterpret_cast<const CUtensorMap*>(&m_out), q);
}

}  // namespace

// True (and the launch issued, its result in *err) when the transform is one TMA can express: 16-byte-aligned bases
// and strides, at least ~1 MB to move, and either the same fastest dim on both sides (elements of 2 or 4 bytes) or two
// different fastest dims of 16-bit elements. dims / xs / ys: the transform's logical dims with input and output
// element strides.
bool launch_permute_tma(const PermuteParams& p, uint32_t* status, cudaStream_t st, cudaError_t* err) {
  *err = cudaSuccess;
  // dims by output stride, fastest first
  int idx[5], n = 0;
  for (int j = 0; j < p.rank; ++j)
    if (p.dims[j] > 1) {
      if (n == 5) return false;
      idx[n++] = j;
    }
  if (n < 2) return false;
  std::sort(idx, idx + n, [&](int a, int b) { return p.ys[a] < p.ys[b]; });
  if (p.ys[idx[0]] != 1) return false;
  const int es = p.esize;
  const bool rows = p.xs[idx[0]] == 1;
  if (!rows) {
    // tiles form: move the input's fastest dim to the front, the output's fastest dim behind it
    if (es != 2) return false;
    int xi = -1;
    for (int k = 1; k < n; ++k)
      if (p.xs[idx[k]] == 1) xi = k;
    if (xi < 0) return false;
    const int o = idx[0], i = idx[xi];
    for (int k = xi; k > 1; --k) idx[k] = idx[k - 1];
    idx[0] = i;
    idx[1] = o;
  }
  int64_t total_el = 1;
  for (int k = 0; k < n; ++k) total_el *= p.dims[idx[k]];
  if (total_el * es < (int64_t(1) << 20)) return false;
  const char* x = static_cast<const char*>(p.x) + p.x_offset * es;
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(p.y) & 15)) return false;
  uint64_t dims[5], xs_b[5], ys_b[5];
  uint32_t box[5];
  for (int d = 0; d < 5; ++d) { dims[d] = 1; xs_b[d] = ys_b[d] = 16; box[d] = 1; }
  for (int k = 0; k < n; ++k) {
    dims[k] = (uint64_t)p.dims[idx[k]];
    xs_b[k] = (uint64_t)p.xs[idx[k]] * es;
    ys_b[k] = (uint64_t)p.ys[idx[k]] * es;
    const bool fast_in = k == 0, fast_out = rows ? k == 0 : k == 1;
    if (!fast_in && ((xs_b[k] & 15) || xs_b[k] >= (uint64_t(1) << 40))) return false;
    if (!fast_out && ((ys_b[k] & 15) || ys_b[k] >= (uint64_t(1) << 40))) return false;
  }
  const TmaCfg& cfg = tma_cfg();
  PermTma q{};
  q.status = status;
  TensorMapStorage m_in, m_out;
  if (rows) {
    if ((dims[0] * es) & 15) return false;
    // box: the fast dim (at most 256 elements a box) x as many rows of the next dim as the box holds
    const uint32_t box_bytes = uint32_t(cfg.box_kb_a) * 1024;
    box[0] = (uint32_t)std::min<uint64_t>(dims[0], 256);
    while ((box[0] * es) & 15) --box[0];
    box[1] = std::max<uint32_t>(1, (uint32_t)std::min<uint64_t>(std::min<uint64_t>(dims[1], 256), box_bytes / (box[0] * es)));
    q.stages = cfg.stages_a;
    q.stage_bytes = box_bytes;
    q.box_bytes = box[0] * box[1] * es;
    if (encode_tensor_map_plain(&m_in, x, es, dims, xs_b, box) != 0 || encode_tensor_map_plain(&m_out, p.y, es, dims, ys_b, box) != 0)
      return false;
  } else {
    box[0] = box[1] = 64;
    q.stages = cfg.stages_b;
    q.stage_bytes = q.box_bytes = 64 * 64 * 2;
    // the output map in its own order: O fastest, then I
    uint64_t odims[5], ostr[5];
    for (int d = 0; d < 5; ++d) { odims[d] = dims[d]; ostr[d] = ys_b[d]; }
    std::swap(odims[0], odims[1]);
    std::swap(ostr[0], ostr[1]);
    if (encode_tensor_map_plain(&m_in, x, es, dims, xs_b, box, true) != 0 ||
        encode_tensor_map_plain(&m_out, p.y, es, odims, ostr, box, true) != 0)
      return false;
  }
  int64_t total = 1;
  for (int d = 0; d < 5; ++d) {
    q.box[d] = (int)box[d];
    q.n_box[d] = (int)((dims[d] + box[d] - 1) / box[d]);
    total *= q.n_box[d];
  }
  if (total >= (int64_t(1) << 31)) return false;
  q.total = (int)total;
  *err = rows ? launch_form<false>(m_in, m_out, q, cfg.warps_a, cfg.ctas_a, st) : launch_form<true>(m_in, m_out, q, cfg.warps_b, cfg.ctas_b, st);
  return true;
}

}  // namespace fluid
