// Internal host-side data model of the planner and executor (not part of the C-ABI).
#pragma once

#include <array>
#include <cstdint>
#include <cstring>
#include <limits>
#include <mutex>
#include <string>
#include <vector>

#include "fluid.h"
#include "kernels.h"

namespace fluid {

constexpr double kInf = std::numeric_limits<double>::infinity();

struct TensorDesc {
  int dtype = FLUID_F32;
  int rank = 0;
  int64_t dims[FLUID_MAX_RANK] = {1, 1, 1, 1, 1};
  int kind = FLUID_ACT;
  int64_t numel() const {
    int64_t n = 1;
    for (int i = 0; i < rank; ++i) n *= dims[i];
    return n;
  }
  int64_t esize() const { return dtype == FLUID_BF16 ? 2 : 4; }
};

struct OpDesc {
  int kind = 0;
  std::vector<int> ins, outs;
  fluid_op_attrs attrs{};
};

using Perm = std::array<int8_t, FLUID_MAX_RANK>;

inline Perm identity_perm() { return Perm{0, 1, 2, 3, 4}; }

// Element strides per logical dim for a dense tensor stored with dims ordered `perm`
// (slowest to fastest).
inline void strides_of(const TensorDesc& t, const Perm& perm, int64_t* st) {
  int64_t run = 1;
  for (int i = t.rank - 1; i >= 0; --i) {
    st[perm[i]] = run;
    run *= t.dims[perm[i]];
  }
}

// A planning node: one graph op, or several folded into one kernel step.
enum NodeKind { N_EMBED, N_GEMM, N_NORM, N_SOFTMAX, N_ROPE, N_ELTWISE, N_TRANSPOSE, N_SELECT, N_ATTN, N_ATTN_DECODE };
enum GemmKind { G_LINEAR, G_QK, G_PV };

struct Node {
  int kind = 0;
  std::vector<int> ops;        // graph op ids folded into this node, first = anchor
  std::vector<int> ins, outs;  // distinct external tensors, inputs in role order
  // role-tagged tensor ids (-1 = absent)
  int a = -1, b = -1, bias = -1, res = -1, out = -1, gamma = -1, beta = -1, pos = -1, v = -1, kc = -1, vc = -1, pos_off = -1;
  int gemm_kind = G_LINEAR, contract = 1, act = ACT_NONE, causal = CAUSAL_NONE;
  double scale = 1.0, eps = 1e-5, rope_base = 10000.0;
  int elt = ELT_ADD, rms = 0, rope_interleaved = 0, sm_causal = 0, rope_fused = 0;
  int perm[8] = {0, 1, 2, 3, 4, 5, 6, 7};
};

// One executable step: a kernel id plus the tensors it touches; launch parameters are derived
// from the plan's layouts when the plan is finalised.
struct Step {
  int kernel = 0;
  int variant = 0;
  int node = -1;            // first (or only) planning node of this step
  std::vector<int> nodes;   // all nodes run by this step (grouped sibling GEMMs: up to 3)
  double cost = 0, flops = 0, bytes = 0;
  // launch payloads (one of these is used, by kernel id)
  GemmParams gemm{};
  GemmTcHost tc{};
  GemmParams gemm_x[2]{};   // groups 1 and 2 of a grouped GEMM step
  GemmTcHost tc_x[2]{};
  int x_ptr[2][3] = {{-1, -1, -1}, {-1, -1, -1}};  // tensor ids of B, C, bias for groups 1 and 2
  int split_k = 1;          // GEMM steps with few tiles cut their k range across CTAs
  int cluster_k = 0;        // >1: the cut runs as one thread-block cluster per output tile (no scratch)
  int swiglu = 0;           // 1: nodes = {gate GEMM, up GEMM, SiLU(gate) * up}: one CTA-pair launch, gate and up never stored
  RopeFreq rope_freq{};     // frequency table of the fused rotary embeddings
  int rope_fused = 0;       // >0: that many trailing nodes are the rotary embeddings of this step's first projections (CTA-pair GEMM epilogue); the unrotated projections are never stored
  int norm_fused = 0;       // 1: the last node is the RMS normalisation that feeds every GEMM of the step (few-row kernel only); its output is never stored
  float norm_eps = 0.f;
  int norm_x_f32 = 0;
  // An RMS normalisation split across two CTA-pair GEMM steps: the step that writes the residual stream (nrm_emit) also
  // writes bf16(x * gain) and per-slab sums of squares into a scratch slice that lives until the step that reads the
  // normalised tensor (nrm_pre: its last node is the normalisation; its GEMMs take the scratch as A and scale their rows).
  int nrm_emit = 0, nrm_pre = 0;
  int nrm_node = -1;        // the normalisation's node (both steps)
  int nrm_record = -1;      // the scratch slice of bf16(x * gain) (both steps)
  int nrm_ss_record = -1;   // the scratch slice of the slabs' sums of squares (both steps)
  int64_t scratch_bytes = 0;
  int scratch_record = -1;  // arena slice holding the split-K partial tiles (alive during this step only)
  NormParams norm{};
  SoftmaxParams softmax{};
  RopeParams rope{};
  EltParams elt{};
  PermuteParams permute{};
  EmbedParams embed{};
  AttnParams attn{};
  AttnHost attn_host{};
  AttnDecodeParams attn_dec{};
  // tensor ids whose device addresses fill the payload's pointer slots
  int t_ptr[8] = {-1, -1, -1, -1, -1, -1, -1, -1};
  int t_narrow[8] = {0, 0, 0, 0, 0, 0, 0, 0};  // 1: bind the bf16 twin of an fp32-held tensor
};

struct ArenaRecord {
  int root = -1;  // root tensor id
  int64_t bytes = 0;
  int first = 0, last = 0;
  int64_t offset = -1;
  int id = -1;    // root, or root + number of tensors for a twin
  int twin = 0;   // 1: the bf16 copy of a tensor whose primary storage is fp32
  int step = -1;  // >= 0: per-step scratch (root is -1)
};

}  // namespace fluid

struct fluid_graph_s {
  std::vector<fluid::TensorDesc> tensors;
  std::vector<fluid::OpDesc> ops;
};

struct fluid_plan_s {
  fluid_graph_s graph;  // private copy
  fluid_plan_options opts{};
  std::vector<std::vector<fluid::Perm>> cands;  // per tensor
  std::vector<fluid::Node> nodes;               // in linear order
  std::vector<int> node_of_op;
  std::vector<std::vector<int>> sequences;      // node ids
  std::vector<int> layout;                      // per tensor: candidate index
  std::vector<int> alias_root;                  // per tensor: root tensor id
  std::vector<int> storage_root;                // per tensor: the tensor whose arena record holds it (alias root, or further the operand an in-place step wrote over)
  std::vector<int> folded;                      // per tensor: 1 if removed by fusion
  std::vector<int> op_variant;                  // per graph op: the caller's variant request (copy of opts.op_variant)
  std::vector<int> node_variant;                // per node: the variant rated best under the final layouts (0: none)
  int not_runnable_op = -1;                     // a caller's cost function chose layouts no kernel runs for this op: the plan is kept for inspection, fluid_run refuses it
  std::vector<fluid::Step> steps;
  std::vector<fluid::ArenaRecord> records;
  std::vector<int> record_of;                   // per tensor (root): index in records or -1
  std::vector<int> twin_record_of;              // per tensor: index of its bf16 twin slice or -1
  std::vector<char> wide;                       // per tensor: 1 = held in fp32 although declared bf16
  std::vector<int> first_step, last_step;       // per tensor
  std::vector<const void*> const_ptr;           // per tensor
  std::vector<int> input_slot, output_slot;     // per tensor: index in inputs/outputs or -1
  size_t arena_bytes = 0, naive_bytes = 0, live_bound = 0;
  double cost = 0, canonical_cost = 0;
  // executor state: tensor maps are encoded for one set of base addresses and re-encoded when
  // any of them changes
  std::mutex mu;
  std::vector<const void*> bound_key;
  bool maps_valid = false;
};

namespace fluid {
void set_error(const char* fmt, ...);
int finalize_steps(fluid_plan_s* p);               // executor-side: derive launch payloads
double node_cost(const fluid_plan_s* p, const Node& n, const int* lo);   // built-in table; +infinity = no kernel
int pack_constant_launch(const fluid_plan_s* p, int tid, const void* src, void* dst, void* stream);
double node_cost(const fluid_plan_s* p, const Node& n, const int* layout_of /*per tensor*/);
bool transpose_is_alias(const fluid_plan_s* p, const Node& n, const int* layout_of);
// Lower a GEMM-like node under the given layouts; false if the node cannot be expressed.
bool lower_gemm(const fluid_plan_s* p, const Node& n, const int* layout_of, GemmParams* gp);
bool gemm_tc_eligible(const fluid_plan_s* p, const GemmParams& gp, GemmTcHost* tc, int variant = 0);
// Implementation variants of a tensor-core GEMM node (codes of kernels.h), their analytic rating, and the choice.
std::vector<int> gemm_tc_variants(const fluid_plan_s* p, const GemmParams& g, int n_group);
double gemm_tc_variant_cost(const GemmParams& g, const GemmTcHost& tc, int n_group);
int gemm_variant_of(const fluid_plan_s* p, const Node& n);   // requested or rated-best variant of a node, 0 if none
// Lower a fused attention node; false if the layouts cannot be fed to the attention kernel.
bool lower_attn(const fluid_plan_s* p, const Node& n, const int* layout_of, AttnParams* ap, AttnHost* host);
}  // namespace fluid
