// Layout transforms that keep the fastest dim (class A: [B,S,nh,D] -> [B,nh,S,D] and the like) as pure TMA traffic:
// rows of the shared fast dim are gathered by a tiled bulk-tensor load into a ring of shared-memory boxes and leave by
// a tiled bulk-tensor store; no register ever holds the data. Both tensor maps are written in the OUTPUT's dim order
// (the input map with the input's strides), so one coordinate tuple addresses a box on both sides, and the box is
// "R rows of the next-fastest output dim": the store is one dense run of R rows, the load a gather of R row segments.
// One thread per CTA drives the ring: up to kStages - kStoresInFlight loads and kStoresInFlight stores in flight
// (~100 KB per SM), which is what a 16-byte-per-thread register copy could not keep in the air.
// Ragged extents need no code: a load past the end fills zeros, a store past the end is clipped.
// Every wait is bounded; an expired one sets bit 0x400 of the status word and the thread drains and leaves.
#include <cuda.h>

#include <algorithm>

#include "device_utils.cuh"
#include "fluid.h"
#include "kernels.h"

namespace fluid {

namespace {

constexpr int kStages = 8;
constexpr int kStoresInFlight = 2;
constexpr uint32_t kBoxBytes = 16384;
constexpr long long kWaitCycles = 3000000000LL;

struct PermTma {
  int n_box[5];        // boxes along each output dim (fastest first)
  int box[5];          // box extent along each dim
  int total;           // boxes in all
  uint32_t box_bytes;  // bytes one full box brings in
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

__global__ void __launch_bounds__(32, 1)
permute_rows_tma_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_out,
                        const __grid_constant__ PermTma p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 127u) & ~127u;
  const uint32_t bars = base + kStages * kBoxBytes;
  pdl_launch_dependents();
  if (threadIdx.x != 0) return;
  for (int s = 0; s < kStages; ++s)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + 8u * s), "r"(1));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_in)) : "memory");
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_out)) : "memory");
  const int first = blockIdx.x, step = gridDim.x;
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
    const uint32_t bar = bars + 8u * (k % kStages), dst = base + uint32_t(k % kStages) * kBoxBytes;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(p.box_bytes) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&map_in)), "r"(bar), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4])
        : "memory");
  };
  pdl_wait();   // the input comes from the previous step; the output may still be read by it
  for (int k = 0; k < mine && k < kStages; ++k) load(k);
  bool ok = true;
  int landed = 0;   // boxes whose load has been waited for
  for (int k = 0; k < mine; ++k) {
    if (!mbar_wait(bars + 8u * (k % kStages), uint32_t(k / kStages) & 1u)) { ok = false; break; }
    landed = k + 1;
    int c[5];
    coords(k, c);
    asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(&map_out)), "r"(base + uint32_t(k % kStages) * kBoxBytes), "r"(c[0]), "r"(c[1]),
                 "r"(c[2]), "r"(c[3]), "r"(c[4])
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    // the store of box k - kStoresInFlight has read its shared memory: that stage takes the next load
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kStoresInFlight) : "memory");
    const int next = k - kStoresInFlight + kStages;
    if (k >= kStoresInFlight && next < mine) load(next);
  }
  if (!ok) {
    if (p.status) atomicOr(p.status, 0x400u);
    // loads already issued must land before the shared memory goes (each wait bounded)
    const int issued = min(mine, max(kStages, landed - kStoresInFlight + kStages));
    for (int k = landed; k < issued; ++k) mbar_wait(bars + 8u * (k % kStages), uint32_t(k / kStages) & 1u);
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // every store complete before the CTA exits
}

}  // namespace

// True (and the launch issued) when the transform is a row gather TMA can express: same fastest dim on both sides,
// 16-byte-aligned bases and strides, at least ~1 MB to move. dims / xs / ys: the transform's logical dims with input
// and output element strides (PermuteParams); esize 2 or 4.
bool launch_permute_rows_tma(const PermuteParams& p, uint32_t* status, cudaStream_t st, cudaError_t* err) {
  *err = cudaSuccess;
  // dims by output stride, fastest first
  int idx[5], n = 0;
  for (int j = 0; j < p.rank; ++j)
    if (p.dims[j] > 1) idx[n++] = j;
  if (n < 2) return false;
  std::sort(idx, idx + n, [&](int a, int b) { return p.ys[a] < p.ys[b]; });
  if (p.ys[idx[0]] != 1 || p.xs[idx[0]] != 1) return false;   // the fastest dim must be the same on both sides
  const int es = p.esize;
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
    if (k > 0 && ((xs_b[k] & 15) || (ys_b[k] & 15) || xs_b[k] >= (uint64_t(1) << 40) || ys_b[k] >= (uint64_t(1) << 40))) return false;
  }
  if ((dims[0] * es) & 15) return false;
  // box: the whole fast dim (at most 256 elements a box) x as many rows of the next dim as 16 KB hold
  box[0] = (uint32_t)std::min<uint64_t>(dims[0], 256);
  while ((box[0] * es) & 15) --box[0];
  const uint32_t rows = std::max<uint32_t>(1, std::min<uint64_t>(std::min<uint64_t>(dims[1], 256), kBoxBytes / (box[0] * es)));
  box[1] = rows;
  PermTma q{};
  int64_t total = 1;
  for (int d = 0; d < 5; ++d) {
    q.box[d] = (int)box[d];
    q.n_box[d] = (int)((dims[d] + box[d] - 1) / box[d]);
    total *= q.n_box[d];
  }
  if (total >= (int64_t(1) << 31)) return false;
  q.total = (int)total;
  q.box_bytes = box[0] * box[1] * es;
  q.status = status;
  TensorMapStorage m_in, m_out;
  if (encode_tensor_map_plain(&m_in, x, es, dims, xs_b, box) != 0 || encode_tensor_map_plain(&m_out, p.y, es, dims, ys_b, box) != 0)
    return false;
  const size_t smem = size_t(kStages) * kBoxBytes + 8 * kStages + 256;
  static bool attr_done = false;
  if (!attr_done) {
    *err = cudaFuncSetAttribute(permute_rows_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (*err != cudaSuccess) return true;
    attr_done = true;
  }
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned grid = (unsigned)std::min<int64_t>(total, sms);
  *err = launch_k(permute_rows_tma_kernel, grid, 32, smem, st, *reinterpret_cast<const CUtensorMap*>(&m_in),
                  *reinterpret_cast<const CUtensorMap*>(&m_out), q);
  return true;
}

}  // namespace fluid
