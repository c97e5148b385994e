// Launch payloads (plain data, visible to host and device) and launch entry points of the
// sm_100a kernels. Tensor addresses are filled in by the executor from the arena base, the
// bound constants and the caller's input/output pointers.
#pragma once

#include <cmath>
#include <cstdint>

#include <cuda_runtime.h>

namespace fluid {

enum ActKind { ACT_NONE = 0, ACT_GELU_ERF = 1, ACT_GELU_TANH = 2 };
enum CausalKind { CAUSAL_NONE = 0, CAUSAL_SKIP_UPPER = 1, CAUSAL_CLIP_K = 2 };
enum EltKind { ELT_ADD = 0, ELT_MUL = 1, ELT_GELU_ERF = 2, ELT_GELU_TANH = 3, ELT_SILU = 4, ELT_SILU_MUL = 5 };

// C[b, m, n] = epilogue(scale * sum_k A[b, m, k] * B[b, k, n]) with every index split in two
// levels, i = i1 * X0 + i0, and one element stride per level and operand. This one form covers
// LINEAR over any layout of x / W / y (head-major outputs included) and the batched
// attention products over any head layout.
struct GemmParams {
  const void* A;
  const void* B;
  void* C;
  const void* bias;  // indexed by n, dense
  const void* R;     // residual, indexed like C with its own strides
  int dtype;         // FLUID_F32 or FLUID_BF16 (A, B, C, bias, R all share it)
  int M, N, K, batch;
  int M0, N0, K0, B0;  // inner extents of the m, n, k and batch index splits
  int64_t a_s[6];      // strides for b1, b0, m1, m0, k1, k0
  int64_t b_s[6];      // strides for b1, b0, k1, k0, n1, n0
  int64_t c_s[6];      // strides for b1, b0, m1, m0, n1, n0
  int64_t r_s[6];
  int c_f32, r_f32;    // bf16 models only: C / R are held in fp32 (residual-stream tensors)
  float scale;
  int act;
  int causal;  // CAUSAL_SKIP_UPPER: tiles with n > m everywhere are not computed;
               // CAUSAL_CLIP_K: the k loop stops after the tile holding k = m_max
  int has_bias, has_res;
  int b_const;  // B is a constant of the plan (a weight): its loads need not wait for the previous step
  int rope;     // 1: the rotary embedding of the output (heads of 128 columns, pairs (d, d + 64), position = row % rope_S) runs in the epilogue
  int rope_S;   // rows per sequence
  // An RMS normalisation split across two tensor-core steps (CTA-pair form). The step that produces the residual
  // stream x (this GEMM's fp32 output) also writes bf16(x * gain) and, per row and 128-column slab, the sum of x^2 ...
  void* nrm_out;          // bf16, same element offsets as C
  const void* nrm_gamma;  // bf16 gain, indexed by n
  float* nrm_ss;          // [M][N / 128] sums of squares
  // ... and the steps that read the normalised tensor take bf16(x * gain) as their A operand and scale their
  // accumulator rows by 1 / rms, formed from the slabs in slab order: (x * gain / rms) . W = ((x * gain) . W) / rms.
  const float* row_ss;    // [M][row_slabs]
  int row_slabs;
  float row_inv_n, row_eps;   // 1 / (elements of a normalised row), the normalisation's epsilon
};

// Host-side description of the two TMA tensor maps of a tensor-core GEMM step.
struct TmaOperand {
  int rank;
  uint64_t dims[5];     // elements, fastest first
  uint64_t strides[5];  // elements; strides[0] == 1
  uint32_t box[5];
  int sel[5];           // which index feeds each coordinate: 0 k0, 1 k1, 2 r0, 3 r1, 4 b0, 5 b1
  int k0, r0, b0;       // inner extents used to split the k, row and batch indices
  int mn_major;         // 1: the row (m or n) index is the contiguous one
};

struct GemmTcCfg {
  int bn;               // tile width (64, 128 or 256); tile height is 128, depth 64
  int stages;
  int a_mn_major, b_mn_major;
  int a_sel[5], b_sel[5];
  int a_k0, a_r0, a_b0, b_k0, b_r0, b_b0;
  int a_rank, b_rank;
  int b_box_rows;       // rows of one TMA box of a K-major B tile (bn, or 128 when a CTA pair shares a 256-wide tile)
  int pair;             // 1: the step qualifies for the CTA-pair kernel (two CTAs, one 256 x 256 tile, tcgen05 cta_group::2)
  int no_cluster;       // 1: the step was asked to run without the cluster split-K form
  int want_cluster;     // 1: the step was asked to run as clusters that split k (refused at lowering if the shape does not qualify)
};

// Implementation variants of a tensor-core GEMM step (the counterpart of the paper's loop orders: same numbers, different
// time). code = form | tile_n << 4; 0 = chosen by the built-in rules.
//   form 1: one CTA per 128 x tile_n tile (persistent, tile_n 64 / 128 / 256)
//   form 2: a pair of CTAs per 256 x 256 tile (tcgen05 cta_group::2; tile_n 256)
//   form 3: a thread-block cluster per 128 x tile_n tile that splits k (tile_n 64 / 128; few-tile steps only)
constexpr int GV_AUTO = 0, GV_SINGLE = 1, GV_PAIR = 2, GV_CLUSTER = 3;
inline int gemm_variant_code(int form, int bn) { return form | (bn << 4); }
inline int gemm_variant_form(int code) { return code & 15; }
inline int gemm_variant_bn(int code) { return code >> 4; }

struct alignas(64) TensorMapStorage {
  unsigned char bytes[128];
};

struct GemmTcHost {
  int eligible;
  TmaOperand a, b;
  GemmTcCfg cfg;
  TensorMapStorage map_a, map_b;
};

struct NormParams {
  const void* x;
  const void* res;    // optional second addend (x + res is normalised)
  const void* gamma;
  const void* beta;   // null for RMSNorm
  void* y_lo;         // output in the model dtype (may be null when only y_hi is wanted)
  float* y_hi;        // bf16 models: optional fp32 copy of the output (residual stream)
  int dtype;
  int x_f32, res_f32; // bf16 models: x / res are held in fp32
  int rows, width;
  float eps;
  int rms;
};

struct SoftmaxParams {
  const void* x;
  void* y;
  int dtype;
  int64_t rows;
  int n;              // row length
  int rows_per_mat;   // causal: row index inside its matrix = row % rows_per_mat
  float scale;
  int causal;
  int zero_block;     // causal: 0 = zeros are written to the end of the row; else only up to the next
                      // multiple of zero_block past the diagonal (the consumer reads no further)
};

// Rotary frequencies base^(-2i/D) of the first 64 pairs, computed once on the host in double and handed over as a pair of
// floats (hi + lo carries 48 bits); pairs beyond 64 are computed on the device from log2_base (head dims above 128).
struct RopeFreq {
  double log2_base;
  float hi[64], lo[64];
};
inline void rope_freq_fill(RopeFreq& t, double base, int D) {
  t.log2_base = std::log2(base);
  for (int i = 0; i < 64; ++i) {
    const double f = std::exp2(-2.0 * i / D * t.log2_base);
    t.hi[i] = (float)f;
    t.lo[i] = (float)(f - (double)t.hi[i]);
  }
}

struct RopeParams {
  const void* x;
  void* y;
  int dtype;
  int dims[4];        // B, S, nh, D
  int64_t st[4];      // element strides of x and y (same layout) per logical dim
  int order[4];       // logical dims, slowest to fastest, in memory
  RopeFreq freq;      // base^(-2i/D), double
  int interleaved;
  const int* pos;     // device: position of row 0 (null = 0)
  int pos_stride;     // 0: one position for the batch, 1: pos[b] per sequence
};

struct EltParams {
  const void* a;
  const void* b;
  void* y;
  int dtype;
  int a_f32, b_f32, y_f32;  // bf16 models: operand held in fp32 (residual-stream tensors)
  int64_t n;
  int op;
};

// y[i0..i4] = x[...] for a dense rank-<=5 tensor; dims are the output's logical dims, xs / ys the
// input / output element strides per output logical dim.
struct PermuteParams {
  const void* x;
  void* y;
  int esize;
  int rank;
  int dims[5];
  int64_t xs[5], ys[5];
  int64_t x_offset;   // elements, added to x
  int x_inner, y_inner;  // output-logical dim that is contiguous in x / in y (-1: none)
  uint32_t* status;      // device status word for the TMA form's bounded waits (may be null)
};

struct EmbedParams {
  const int* ids;
  const void* tok;
  const void* pos;    // optional [P, H]
  const int* pos_off; // optional, device: index of the first position row, for the batch or per sequence
  int pos_off_stride; // 0 or 1
  int P;              // rows of pos
  void* y;
  int dtype;
  int y_f32;          // bf16 models: y is held in fp32
  int tokens, S, H, V;
};

// Fused attention: O[b,h,i,:] = softmax_j(scale * q[b,h,i,:].k[b,h,j,:]) v[b,h,j,:]
struct AttnParams {
  void* O;
  uint32_t* status;
  int B, NH, S, D;
  int64_t o_s[3];       // element strides of b, h, s in O (d contiguous)
  float scale_log2;     // scale * log2(e)
  int causal;
  int k_mn_major;       // K has the sequence index contiguous ([B,nh,D,S] family)
  int v_k_major;        // V has the sequence index contiguous
  int q_sel[5], k_sel[5], v_sel[5];   // tensor-map coordinate feeds: 0 contraction, 2 row, 4 / 5 batch split, 6 zero
  int q_b0, k_b0, v_b0;               // inner extent of each operand's (batch * head) index split
  // plain addressing, for the short-sequence form that reads the operands without tensor maps
  const void *Q, *K, *V;              // bound per run
  int64_t q_s[3], k_s[3], v_s[3];     // element strides of b, h, s
  int rows_d_contiguous;              // Q, K and V all have d contiguous and 16-byte aligned rows
};

// One decoding step against a key/value cache [B, Tmax, NKV, D] (canonical, caller-owned): the new key and
// value become row t = *pos of the caches, the query attends over rows 0..t.
struct AttnDecodeParams {
  int dtype;
  const void *q, *k, *v;  // [B,1,NH,D], [B,1,NKV,D] x 2: d contiguous, strides below
  void *kc, *vc;
  const int* pos;         // device
  int pos_stride;         // 0: one position for the batch, 1: pos[b] per sequence
  void* out;              // [B,1,NH,D]
  uint32_t* status;
  int B, NH, NKV, D, Tmax;
  float scale_log2;       // scale * log2(e)
  int rope;               // 1: q and k arrive unrotated; the step applies the rotary embedding (pairs (d, d + D/2)) at position *pos
  RopeFreq rope_freq;
  int64_t q_sb, q_sh, k_sb, k_sh, v_sb, v_sh, o_sb, o_sh;   // element strides of batch and head
};
// GEMM with at most 16 rows and both operands k-contiguous (bf16): the weights stream through the SM once.
// n_group (1..3) sibling GEMMs that share A and the shapes run as one launch. swiglu (two groups: gate, up): the launch
// writes SiLU(gate) * up to g[0].C and nothing else.
// norm (optional): the RMS normalisation or (M <= 15, no swiglu) LayerNorm in front of the GEMMs runs inside the launch: A is then x (bf16, or fp32 when
// x_f32) with the strides of g[0]'s A operand, and the normalised tensor is never stored.
struct RowsNorm {
  const void* x;
  const void* gamma;
  const void* beta;   // LayerNorm's bias; null for an RMS normalisation
  float eps;
  int x_f32;
};
bool gemm_rows_eligible(const GemmParams& g);
cudaError_t launch_gemm_rows(const GemmParams* g, int n_group, cudaStream_t stream, int swiglu = 0, const RowsNorm* norm = nullptr,
                             uint32_t* status = nullptr);
cudaError_t launch_attn_decode(const AttnDecodeParams& p, cudaStream_t stream);
bool attn_decode_supported(int dtype, int D);

struct AttnHost {
  int eligible;
  TmaOperand q, k, v;
  TensorMapStorage map_q, map_k, map_v;
};

// Launchers: enqueue on `stream`, return the CUDA error of the launch.
cudaError_t launch_gemm_simt(const GemmParams& p, cudaStream_t stream);
// n_group (1..3) GEMMs that share the A operand, the shapes and the tile configuration run as one
// launch (sibling projections such as Q/K/V or gate/up); group i uses g[i] and tc[i].map_b.
// split_k > 1 cuts every output tile's k range into split_k pieces run by different CTAs; `partial`
// then points at n_tiles * split_k * 128 * bn floats of scratch and status[8..63] hold the per-tile
// arrival counters (zero before the launch, left zero after it).
// swiglu (two groups, CTA-pair form only): group 0 is the gate, group 1 the up projection; the launch writes
// SiLU(gate) * up to g[0].C and nothing else.
int encode_tensor_map_plain(TensorMapStorage* out, const void* base, int esize, const uint64_t* dims, const uint64_t* strides_bytes,
                            const uint32_t* box, bool swizzle128 = false);
// Layout transforms as TMA loads and stores (rows gathered when both sides share the fastest dim, 64 x 64 tiles of
// 16-bit elements transposed in shared memory when they do not); false if the transform does not qualify (nothing
// launched).
bool launch_permute_tma(const PermuteParams& p, uint32_t* status, cudaStream_t st, cudaError_t* err);
cudaError_t launch_gemm_tc(const GemmParams* g, const GemmTcHost* tc, int n_group, int split_k, int cluster_k, float* partial,
                           uint32_t* status, cudaStream_t stream, int swiglu = 0, const RopeFreq* rope_freq = nullptr);
// Split factor a GEMM step should use (1 = none) and the scratch it then needs.
int gemm_split_k(const GemmParams& g, const GemmTcHost& tc, int n_group, int64_t* scratch_bytes);
// Cluster size of the cluster split-K form (CTAs of one cluster share an output tile, reduced through
// distributed shared memory; no scratch); 0 if the step runs the persistent kernel.
int gemm_cluster_split(const GemmParams* gs, const GemmTcHost& tc, int n_group);
// True if the step runs on the CTA-pair kernel (two CTAs of a cluster per 256 x 256 tile).
bool gemm_pair_eligible(const GemmParams* gs, const GemmTcHost& tc, int n_group);
bool gemm_tc_describe(const GemmParams& g, GemmTcHost* tc, int variant = 0);
cudaError_t launch_attn_tc(const AttnParams& p, const AttnHost& host, cudaStream_t stream);
// Short sequences (S <= 128) with d contiguous in Q, K and V: one warp per 16 query rows, scores in registers.
bool attn_small_eligible(const AttnParams& p);
cudaError_t launch_attn_small(const AttnParams& p, const AttnHost* host, cudaStream_t stream);
cudaError_t launch_norm(const NormParams& p, cudaStream_t stream);
cudaError_t launch_softmax(const SoftmaxParams& p, cudaStream_t stream);
cudaError_t launch_rope(const RopeParams& p, cudaStream_t stream);
cudaError_t launch_eltwise(const EltParams& p, cudaStream_t stream);
cudaError_t launch_permute(const PermuteParams& p, cudaStream_t stream);
cudaError_t launch_embed(const EmbedParams& p, cudaStream_t stream);

int encode_tensor_map(TensorMapStorage* out, const void* base, const TmaOperand& op);
int sm_count();
bool tc_kernel_available();

}  // namespace fluid
