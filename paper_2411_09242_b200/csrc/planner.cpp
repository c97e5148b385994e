// fluid_plan(): the layout-and-memory planner (host only).
//
// Pipeline, in the order the paper's compiler applies it (Sec. "Implementation", "Compiler"):
// fusion -> linear sequence -> layout reschedule -> memory plan.
//   linearise        topological order, smallest ready op id first
//   build_nodes      epilogue / elementwise fusion into planning nodes
//   split            Algorithms 1 and 2: longest sequence, remove, recurse on connected remains
//   dp_on_sequence   Eq. 1 / Algorithm 3: cheapest layout per edge of a sequence
//   merge            majority vote over conflicting proposals, losers re-optimise
//   lower            elided TRANSPOSEs become aliases, nodes become kernel steps
//   liveness + Greedy-by-Size  Algorithm 4
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <map>
#include <new>
#include <set>

#include "fluid_internal.h"

namespace fluid {

// ---- analytic B200 cost table (the default eval()) ------------------------------------------
static constexpr double kBw = 6.0e12;        // bytes/s a streaming kernel sustains
static constexpr double kTcPeak = 1.3e15;    // bf16 tensor-core flop/s under sustained load
static constexpr double kSimtPeak = 1.5e13;  // flop/s of the SIMT GEMM
static constexpr double kLaunch = 2.5e-6;    // per-step launch + drain

static const Perm& perm_of(const fluid_plan_s* p, int t, const int* layout_of) { return p->cands[t][layout_of[t]]; }

static bool same_perm(const fluid_plan_s* p, int a, int b, const int* lo) {
  const TensorDesc& ta = p->graph.tensors[a];
  const Perm &pa = perm_of(p, a, lo), &pb = perm_of(p, b, lo);
  for (int i = 0; i < ta.rank; ++i)
    if (pa[i] != pb[i]) return false;
  return true;
}

static bool is_identity(const fluid_plan_s* p, int t, const int* lo) {
  const Perm& pm = perm_of(p, t, lo);
  for (int i = 0; i < p->graph.tensors[t].rank; ++i)
    if (pm[i] != i) return false;
  return true;
}

static double tbytes(const fluid_plan_s* p, int t) {
  const TensorDesc& d = p->graph.tensors[t];
  return double(d.numel()) * double(d.esize());
}

bool transpose_is_alias(const fluid_plan_s* p, const Node& n, const int* lo) {
  const TensorDesc &x = p->graph.tensors[n.a], &y = p->graph.tensors[n.out];
  if (y.kind == FLUID_OUTPUT) return false;  // the caller's buffer must really be written
  int64_t sx[FLUID_MAX_RANK], sy[FLUID_MAX_RANK];
  strides_of(x, perm_of(p, n.a, lo), sx);
  strides_of(y, perm_of(p, n.out, lo), sy);
  for (int j = 0; j < y.rank; ++j)
    if (y.dims[j] > 1 && sy[j] != sx[n.perm[j]]) return false;
  return true;
}

// Split `count` consecutive logical dims starting at `first` into (outer, inner) levels.
static bool two_level(const TensorDesc& t, const int64_t* st, int first, int count, int* x0, int64_t* s1,
                      int64_t* s0, int64_t* total) {
  if (count == 1) {
    *x0 = (int)t.dims[first];
    *s1 = 0;
    *s0 = st[first];
    *total = t.dims[first];
    return true;
  }
  if (count == 2) {
    *x0 = (int)t.dims[first + 1];
    *s1 = st[first];
    *s0 = st[first + 1];
    *total = t.dims[first] * t.dims[first + 1];
    return true;
  }
  return false;
}

bool lower_gemm(const fluid_plan_s* p, const Node& n, const int* lo, GemmParams* gp) {
  const auto& T = p->graph.tensors;
  const TensorDesc &ta = T[n.a], &tb = T[n.b], &tc = T[n.out];
  int64_t sa[FLUID_MAX_RANK], sb[FLUID_MAX_RANK], sc[FLUID_MAX_RANK], sr[FLUID_MAX_RANK];
  strides_of(ta, perm_of(p, n.a, lo), sa);
  strides_of(tb, perm_of(p, n.b, lo), sb);
  strides_of(tc, perm_of(p, n.out, lo), sc);
  if (n.res >= 0) strides_of(T[n.res], perm_of(p, n.res, lo), sr);
  GemmParams g{};
  g.dtype = tc.dtype;
  int64_t M, N, K, tot;
  int x0;
  if (n.gemm_kind == G_LINEAR) {
    const int c = n.contract, mc = ta.rank - c, nc = tb.rank - c;
    if (!two_level(ta, sa, 0, mc, &g.M0, &g.a_s[2], &g.a_s[3], &M)) return false;
    if (!two_level(ta, sa, mc, c, &g.K0, &g.a_s[4], &g.a_s[5], &K)) return false;
    if (!two_level(tb, sb, 0, c, &x0, &g.b_s[2], &g.b_s[3], &tot)) return false;
    if (!two_level(tb, sb, c, nc, &g.N0, &g.b_s[4], &g.b_s[5], &N)) return false;
    if (!two_level(tc, sc, 0, mc, &x0, &g.c_s[2], &g.c_s[3], &tot)) return false;
    if (!two_level(tc, sc, mc, nc, &x0, &g.c_s[4], &g.c_s[5], &tot)) return false;
    if (n.res >= 0) {
      two_level(T[n.res], sr, 0, mc, &x0, &g.r_s[2], &g.r_s[3], &tot);
      two_level(T[n.res], sr, mc, nc, &x0, &g.r_s[4], &g.r_s[5], &tot);
    }
    g.batch = 1;
    g.B0 = 1;
  } else {
    // rank-4 operands [B, nh, rows, cols]: batch = (B, nh)
    g.batch = int(ta.dims[0] * ta.dims[1]);
    g.B0 = (int)ta.dims[1];
    g.a_s[0] = sa[0]; g.a_s[1] = sa[1]; g.a_s[2] = 0; g.a_s[3] = sa[2]; g.a_s[4] = 0; g.a_s[5] = sa[3];
    g.b_s[0] = sb[0]; g.b_s[1] = sb[1]; g.b_s[2] = 0; g.b_s[3] = sb[2]; g.b_s[4] = 0; g.b_s[5] = sb[3];
    g.c_s[0] = sc[0]; g.c_s[1] = sc[1]; g.c_s[2] = 0; g.c_s[3] = sc[2]; g.c_s[4] = 0; g.c_s[5] = sc[3];
    M = ta.dims[2];
    K = ta.dims[3];
    N = tb.dims[3];
    g.M0 = (int)M; g.K0 = (int)K; g.N0 = (int)N;
    if (n.res >= 0) return false;
  }
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return false;
  g.M = (int)M; g.N = (int)N; g.K = (int)K;
  g.scale = (float)n.scale;
  g.act = n.act;
  g.causal = n.causal;
  g.has_bias = n.bias >= 0;
  g.has_res = n.res >= 0;
  *gp = g;
  return true;
}

// ---- TMA operand description for the tensor-core GEMM -------------------------------------------
// An operand is a set of (extent, stride) levels: row (r1, r0), contraction (k1, k0), batch
// (b1, b0). Levels whose strides chain are merged; one level must be contiguous (k0: "K-major",
// r0: "MN-major"); the rest must be 16-byte multiples; tiles may not straddle an unmerged level.
static bool build_tma_operand(int64_t R, int R0, const int64_t* rs, int64_t K, int K0, const int64_t* ks,
                              int64_t BATCH, int B0, const int64_t* bs, int tile_rows, TmaOperand* o) {
  struct Lvl { int64_t n1, n0, s1, s0; bool merged; };
  auto mk = [](int64_t total, int x0, const int64_t* s) {
    Lvl l;
    l.n0 = x0;
    l.n1 = total / x0;
    l.s1 = s[0];
    l.s0 = s[1];
    l.merged = false;
    if (l.n1 == 1) {
      l.merged = true;
    } else if (l.n0 == 1) {
      l.n0 = l.n1; l.s0 = l.s1; l.n1 = 1; l.merged = true;
    } else if (l.s1 == l.n0 * l.s0) {
      l.n0 = total; l.n1 = 1; l.merged = true;
    }
    return l;
  };
  Lvl r = mk(R, R0, rs), k = mk(K, K0, ks), b = mk(BATCH, B0, bs);
  const bool k_major = (k.n0 == 1 && k.n1 == 1) ? (r.s0 != 1) : (k.s0 == 1);
  const bool mn_major = !k_major && (r.s0 == 1 || (r.n0 == 1 && r.n1 == 1));
  if (!k_major && !mn_major) return false;
  if (k.n0 * k.n1 == 1 && !k_major) { /* degenerate K = 1 handled as MN-major */ }
  auto aligned = [](int64_t n, int64_t s) { return n == 1 || (s % 8 == 0); };
  if (k_major) {
    if (!(k.s0 == 1 || k.n0 == 1)) return false;
    if (!aligned(k.n1, k.s1) || !aligned(r.n0, r.s0) || !aligned(r.n1, r.s1)) return false;
    if (!k.merged && k.n0 % 64 != 0) return false;
    if (!r.merged && r.n0 % tile_rows != 0) return false;
  } else {
    if (!aligned(r.n1, r.s1) || !aligned(k.n0, k.s0) || !aligned(k.n1, k.s1)) return false;
    if (!r.merged && r.n0 % 64 != 0) return false;
    if (!k.merged && k.n0 % 64 != 0) return false;
  }
  if (!aligned(b.n0, b.s0) || !aligned(b.n1, b.s1)) return false;
  TmaOperand t{};
  t.mn_major = mn_major ? 1 : 0;
  t.k0 = (int)k.n0; t.r0 = (int)r.n0; t.b0 = (int)b.n0;
  int d = 0;
  auto push = [&](int64_t n, int64_t s, uint32_t box, int sel) {
    t.dims[d] = (uint64_t)n; t.strides[d] = (uint64_t)s; t.box[d] = box; t.sel[d] = sel; ++d;
  };
  if (k_major) {
    push(k.n0, 1, 64, 0);
    if (k.n1 > 1) push(k.n1, k.s1, 1, 1);
    push(r.n0, r.n0 == 1 ? 8 : r.s0, (uint32_t)tile_rows, 2);
  } else {
    push(r.n0, 1, 64, 2);
    if (r.n1 > 1) push(r.n1, r.s1, 1, 3);
    push(k.n0, k.n0 == 1 ? 8 : k.s0, 64, 0);
    if (k.n1 > 1) push(k.n1, k.s1, 1, 1);
  }
  if (k_major && r.n1 > 1) {
    if (d >= 5) return false;
    push(r.n1, r.s1, 1, 3);
  }
  if (b.n0 > 1) {
    if (d >= 5) return false;
    push(b.n0, b.s0, 1, 4);
  }
  if (b.n1 > 1) {
    if (d >= 5) return false;
    push(b.n1, b.s1, 1, 5);
  }
  if (d > 5) return false;
  t.rank = d;
  for (int q = d; q < 5; ++q) { t.dims[q] = 1; t.strides[q] = 8; t.box[q] = 1; t.sel[q] = 6; }
  // contiguity of the fastest level
  if (t.dims[0] > 1 && t.strides[0] != 1) return false;
  *o = t;
  return true;
}

bool gemm_tc_eligible(const fluid_plan_s* p, const GemmParams& g, GemmTcHost* tc, int variant) {
  GemmTcHost h{};
  h.eligible = 0;
  *tc = h;
  if (p->opts.gemm_path == 1) return false;
  if (variant && gemm_tc_describe(g, tc, variant)) return true;   // a variant the shape cannot take falls back to the rules
  return gemm_tc_describe(g, tc, 0);
}

// Tile configuration and TMA operand descriptions of a bf16 GEMM for the tensor-core kernel;
// false if its operands cannot be expressed as tensor maps.
bool gemm_tc_describe(const GemmParams& g, GemmTcHost* tc, int variant) {
  GemmTcHost h{};
  h.eligible = 0;
  *tc = h;
  if (!tc_kernel_available() || g.dtype != FLUID_BF16) return false;
  if (g.K < 8) return false;
  const int form = gemm_variant_form(variant), want_bn = gemm_variant_bn(variant);
  if (variant) {
    if (want_bn != 64 && want_bn != 128 && want_bn != 256 && !(want_bn == 192 && form == GV_PAIR)) return false;
    if (form == GV_PAIR && ((want_bn != 256 && want_bn != 192) || g.causal != CAUSAL_NONE || g.M % 256 != 0)) return false;
    if (form == GV_CLUSTER && (want_bn > 128 || g.causal != CAUSAL_NONE)) return false;
    if (form < GV_SINGLE || form > GV_CLUSTER) return false;
  }
  int bn = 128;
  if (variant) bn = want_bn;
  else if (g.N <= 64) bn = 64;
  else {
    const int64_t tiles256 = int64_t((g.M + 127) / 128) * ((g.N + 255) / 256) * g.batch;
    const int64_t tiles64 = int64_t((g.M + 127) / 128) * ((g.N + 63) / 64) * g.batch;
    if (g.N >= 256 && tiles256 >= 74) bn = 256;
    // few tiles and a k range worth cutting: the step will run as clusters that split k (the tensor core
    // spends the same time on a 128 x 64 x 16 instruction as on a 128 x 128 x 16 one, and the narrower
    // tile halves what the cluster has to exchange), if four CTAs per tile still fit one wave
    else if (g.causal == CAUSAL_NONE && g.K >= 256 && tiles64 * 4 <= 148) bn = 64;
  }
  const int64_t a_rs[2] = {g.a_s[2], g.a_s[3]}, a_ks[2] = {g.a_s[4], g.a_s[5]}, a_bs[2] = {g.a_s[0], g.a_s[1]};
  const int64_t b_rs[2] = {g.b_s[4], g.b_s[5]}, b_ks[2] = {g.b_s[2], g.b_s[3]}, b_bs[2] = {g.b_s[0], g.b_s[1]};
  if (!build_tma_operand(g.M, g.M0, a_rs, g.K, g.K0, a_ks, g.batch, g.B0, a_bs, 128, &h.a)) return false;
  // an unmerged n level narrower than the tile would be straddled: shrink the tile first
  // A 256-wide tile over an even number of 128-row tiles can be shared by a pair of CTAs (each loads half
  // of the B tile: its TMA box is then 128 rows, which the single-CTA kernel fetches as two boxes).
  int b_box = bn;
  while (true) {
    b_box = (bn == 256 && g.causal == CAUSAL_NONE && g.M % 256 == 0 && form != GV_SINGLE) ? 128 : (bn == 192 ? 96 : bn);
    if (build_tma_operand(g.N, g.N0, b_rs, g.K, g.K0, b_ks, g.batch, g.B0, b_bs, b_box, &h.b)) break;
    if (bn == 64 || variant) return false;   // a requested tile width is not traded for a narrower one
    bn /= 2;
  }
  // a pair's 192-wide tile (96 columns of B per CTA: one box of a k-contiguous operand; 64-column boxes do not add up to it)
  if (bn == 192 && h.b.mn_major) return false;
  h.cfg.b_box_rows = b_box;
  h.cfg.pair = ((bn == 256 && b_box == 128) || (bn == 192 && b_box == 96)) ? 1 : 0;
  if (form == GV_PAIR && !h.cfg.pair) return false;
  h.cfg.no_cluster = (form == GV_SINGLE || form == GV_PAIR) ? 1 : 0;
  h.cfg.want_cluster = form == GV_CLUSTER ? 1 : 0;
  // output / residual vector accesses assume 8-element alignment of every outer stride when the
  // n index is contiguous; otherwise the epilogue falls back to scalar stores (always legal)
  h.cfg.bn = bn;
  h.cfg.stages = bn == 256 ? 4 : (bn == 128 ? 6 : 8);
  h.cfg.a_mn_major = h.a.mn_major;
  h.cfg.b_mn_major = h.b.mn_major;
  for (int i = 0; i < 5; ++i) {
    h.cfg.a_sel[i] = h.a.sel[i];
    h.cfg.b_sel[i] = h.b.sel[i];
  }
  h.cfg.a_k0 = h.a.k0; h.cfg.a_r0 = h.a.r0; h.cfg.a_b0 = h.a.b0;
  h.cfg.b_k0 = h.b.k0; h.cfg.b_r0 = h.b.r0; h.cfg.b_b0 = h.b.b0;
  h.cfg.a_rank = h.a.rank;
  h.cfg.b_rank = h.b.rank;
  h.eligible = 1;
  *tc = h;
  return true;
}

// ---- implementation variants of a tensor-core GEMM step (the paper's "Loop Reordering") ----------------------
// Every (form, tile width) the shape can run with; the order is the tie-break of the rating.
std::vector<int> gemm_tc_variants(const fluid_plan_s* p, const GemmParams& g, int n_group) {
  std::vector<int> out;
  if (p->opts.gemm_path == 1) return out;
  GemmParams gs[3] = {g, g, g};
  for (int form : {GV_PAIR, GV_SINGLE, GV_CLUSTER})
    for (int bn : {256, 192, 128, 64}) {
      GemmTcHost tc;
      const int code = gemm_variant_code(form, bn);
      if (bn == 192 && (form != GV_PAIR || n_group != 1)) continue;   // the pair's second width: plain steps only
      if (bn > 64 && g.N <= bn / 2) continue;            // a tile more than twice as wide as the matrix
      if (!gemm_tc_describe(g, &tc, code)) continue;
      if (form == GV_PAIR && !gemm_pair_eligible(gs, tc, n_group)) continue;
      if (form == GV_CLUSTER && (p->opts.split_k < 0 || gemm_cluster_split(gs, tc, n_group) < 2)) continue;
      out.push_back(code);
    }
  return out;
}

// Analytic rating of one variant, seconds. Measured on B200 and used as constants here: a 128 x N x 16 tensor-core
// instruction issued from shared-memory operands takes about 97 / 107 / 171 cycles for N = 64 / 128 / 256 (the A
// tile's 4 KB are fetched per instruction: ~43 cycles on top of N / 2), a 256 x 256 x 16 instruction of a CTA pair 128
// per CTA; the distributed-shared-memory exchange of a cluster moves ~21 bytes per clock into an SM; an SM stores
// ~32 bytes per clock. Tiles run in waves over the SMs (or SM pairs); the epilogue of a tile overlaps the next
// tile's main loop (two accumulators), so a wave costs the longer of the two and the last epilogue is exposed.
double gemm_tc_variant_cost(const GemmParams& g, const GemmTcHost& tc, int n_group) {
  const double clk = 1.8e9;
  const int sms = 148, bn = tc.cfg.bn;
  const int form = tc.cfg.want_cluster ? GV_CLUSTER : (tc.cfg.pair && tc.cfg.no_cluster ? GV_PAIR : GV_SINGLE);
  const double ksteps = std::ceil(g.K / 64.0);
  const double tiles_m = std::ceil(g.M / 128.0), tiles_n = std::ceil(double(g.N) / bn);
  double tiles = tiles_m * tiles_n * g.batch * n_group;
  if (g.causal != CAUSAL_NONE) tiles *= 0.5 * (1.0 + 1.0 / std::max(1.0, tiles_m));
  const double out_bytes = (g.c_f32 ? 4.0 : 2.0) + (g.has_res ? (g.r_f32 ? 4.0 : 2.0) : 0.0);
  const double act = g.act != ACT_NONE ? 1.6 : 1.0;     // an activation in the epilogue costs issue slots
  const double fill = 1800.0;                           // first loads of a CTA: tensor-map fetch, pipeline ramp
  double cycles;
  if (form == GV_PAIR) {
    const double units = sms / 2, pair_tiles = std::ceil(tiles_m / 2.0) * tiles_n * g.batch * n_group;
    // (a 256 x 192 x 16 instruction holds 96 cycles of tensor-core work per CTA but is paced by the operand fetch:
    // ~108 cycles, from four waves of 192-wide tiles against three of 256-wide ones on 4096 x 3072 x 768)
    const double main = ksteps * 4.0 * (bn == 192 ? 108.0 : 128.0), epi = (128.0 * bn * out_bytes / 32.0 + 128.0 * bn / 256.0 * 10.0) * act;
    cycles = fill + std::ceil(pair_tiles / units) * std::max(main, epi) + epi;
  } else if (form == GV_SINGLE) {
    const double per = bn == 256 ? 171.0 : (bn == 128 ? 107.0 : 97.0);
    const double main = ksteps * 4.0 * per, epi = (128.0 * bn * out_bytes / 32.0 + 128.0 * bn / 256.0 * 10.0) * act;
    cycles = fill + std::ceil(tiles / sms) * std::max(main, epi) + epi;
  } else {
    GemmParams gs[3] = {g, g, g};
    const int sk = std::max(2, gemm_cluster_split(gs, tc, n_group));
    const double per = bn == 128 ? 107.0 : 97.0;
    // Measured on the 128-token encoder shape (per-step event pairs and graph replays with each form forced): with 12
    // k-steps a tile the cluster form is no faster than one CTA per 128 x 64 tile (q / k / v 14.9 vs 13.3 us, FFN1 14.5 vs
    // 14.3, o-proj 12.5 vs 12.5), with 48 it is (FFN2 12.4 vs 22.5): besides the bytes, the exchange costs a round of
    // shared-memory staging and remote completion (~1800 cycles), and a cluster launch, its two barriers and its
    // CTAs' lock-step ~1500 more than the rating's other terms account for (the o-proj, whose fp32-residual epilogue the
    // cluster divides among its CTAs, stays on the cluster form: 13.1 vs 13.3 us).
    const double main = std::ceil(ksteps / sk) * 4.0 * per, exchange = 1800.0 + 128.0 * bn * 4.0 * (sk - 1) / sk / 21.0;
    const double epi = (128.0 * bn * out_bytes / 32.0 + 128.0 * bn / 256.0 * 10.0) * act / sk;
    cycles = fill + main + exchange + epi + 600.0 + 1500.0;
  }
  return cycles / clk;
}

// The variant a GEMM node runs with: the caller's request for its anchor op if there is one, else the rated best
// recorded when the layouts were final, else 0 (the shape rules).
int gemm_variant_of(const fluid_plan_s* p, const Node& n) {
  if (n.kind != N_GEMM || n.ops.empty()) return 0;
  const int op = n.ops[0];
  if (op >= 0 && op < (int)p->op_variant.size() && p->op_variant[op]) return p->op_variant[op];
  const int ni = op < (int)p->node_of_op.size() ? p->node_of_op[op] : -1;
  if (ni >= 0 && ni < (int)p->node_variant.size()) return p->node_variant[ni];
  return 0;
}

bool lower_attn(const fluid_plan_s* p, const Node& n, const int* lo, AttnParams* ap, AttnHost* host) {
  const auto& T = p->graph.tensors;
  const TensorDesc &tq = T[n.a], &tk = T[n.b], &tv = T[n.v], &to = T[n.out];
  if (!tc_kernel_available() || p->opts.gemm_path == 1 || to.dtype != FLUID_BF16) return false;
  const int64_t B = tq.dims[0], NH = tq.dims[1], S = tq.dims[2], D = tq.dims[3];
  if (!(D == 64 || D == 128) || tk.dims[3] != S || tv.dims[2] != S || n.scale <= 0.0) return false;
  int64_t sq[FLUID_MAX_RANK], sk[FLUID_MAX_RANK], sv[FLUID_MAX_RANK], so[FLUID_MAX_RANK];
  strides_of(tq, perm_of(p, n.a, lo), sq);
  strides_of(tk, perm_of(p, n.b, lo), sk);
  strides_of(tv, perm_of(p, n.v, lo), sv);
  strides_of(to, perm_of(p, n.out, lo), so);
  if (so[3] != 1 || so[0] % 8 || so[1] % 8 || so[2] % 8) return false;
  AttnHost h{};
  const int64_t q_rs[2] = {0, sq[2]}, q_ks[2] = {0, sq[3]}, q_bs[2] = {sq[0], sq[1]};
  const int64_t k_rs[2] = {0, sk[3]}, k_ks[2] = {0, sk[2]}, k_bs[2] = {sk[0], sk[1]};
  const int64_t v_rs[2] = {0, sv[3]}, v_ks[2] = {0, sv[2]}, v_bs[2] = {sv[0], sv[1]};
  if (!build_tma_operand(S, (int)S, q_rs, D, (int)D, q_ks, B * NH, (int)NH, q_bs, 64, &h.q) || h.q.mn_major) return false;
  if (!build_tma_operand(S, (int)S, k_rs, D, (int)D, k_ks, B * NH, (int)NH, k_bs, 64, &h.k)) return false;
  if (!build_tma_operand(D, (int)D, v_rs, S, (int)S, v_ks, B * NH, (int)NH, v_bs, 64, &h.v)) return false;
  AttnParams a{};
  a.B = (int)B; a.NH = (int)NH; a.S = (int)S; a.D = (int)D;
  a.o_s[0] = so[0]; a.o_s[1] = so[1]; a.o_s[2] = so[2];
  a.scale_log2 = float(n.scale * 1.4426950408889634);
  a.causal = n.sm_causal;
  a.k_mn_major = h.k.mn_major;
  a.v_k_major = h.v.mn_major ? 0 : 1;
  for (int d = 0; d < 5; ++d) { a.q_sel[d] = h.q.sel[d]; a.k_sel[d] = h.k.sel[d]; a.v_sel[d] = h.v.sel[d]; }
  a.q_b0 = h.q.b0; a.k_b0 = h.k.b0; a.v_b0 = h.v.b0;
  // K is [B,nh,D,S] as an operand and V [B,nh,S,D]: the sequence index is dim 3 of K, dim 2 of V
  for (int d = 0; d < 2; ++d) { a.q_s[d] = sq[d]; a.k_s[d] = sk[d]; a.v_s[d] = sv[d]; }
  a.q_s[2] = sq[2]; a.k_s[2] = sk[3]; a.v_s[2] = sv[2];
  a.rows_d_contiguous = sq[3] == 1 && sk[2] == 1 && sv[3] == 1;
  for (int d = 0; d < 3; ++d)
    if (a.q_s[d] % 8 || a.k_s[d] % 8 || a.v_s[d] % 8) a.rows_d_contiguous = 0;
  h.eligible = 1;
  *ap = a;
  *host = h;
  return true;
}

static double gemm_flops(const GemmParams& g) {
  double f = 2.0 * double(g.batch) * g.M * double(g.N) * g.K;
  if (g.causal != CAUSAL_NONE) f *= 0.5 * (1.0 + 1.0 / std::max(1, g.M));
  return f;
}

static double gemm_bytes(const GemmParams& g) {
  const double es = g.dtype == FLUID_BF16 ? 2.0 : 4.0;
  double a = double(g.batch) * g.M * double(g.K), b = double(g.batch) * g.K * double(g.N),
         c = double(g.batch) * g.M * double(g.N);
  if (g.causal == CAUSAL_SKIP_UPPER) c *= 0.5;
  if (g.causal == CAUSAL_CLIP_K) a *= 0.5;
  return es * (a + b + c * (g.has_res ? 2.0 : 1.0) + (g.has_bias ? g.N : 0));
}

double node_cost(const fluid_plan_s* p, const Node& n, const int* lo) {
  const auto& T = p->graph.tensors;
  switch (n.kind) {
    case N_EMBED: {
      for (int t : n.ins)
        if (!is_identity(p, t, lo)) return kInf;
      if (!is_identity(p, n.out, lo)) return kInf;
      return kLaunch + 2.0 * tbytes(p, n.out) / kBw;
    }
    case N_GEMM: {
      GemmParams g;
      if (!lower_gemm(p, n, lo, &g)) return kInf;
      if (n.bias >= 0 && !is_identity(p, n.bias, lo)) return kInf;
      if (n.res >= 0) {
        for (int i = 0; i < 6; ++i)
          if (g.r_s[i] != g.c_s[i]) return kInf;
      }
      GemmTcHost tc;
      const double fl = gemm_flops(g), by = gemm_bytes(g);
      // a handful of rows with k contiguous on both sides: the weight streams through registers once
      if (p->opts.gemm_path == 0 && gemm_rows_eligible(g)) return kLaunch + 0.95 * by / kBw;
      if (gemm_tc_eligible(p, g, &tc)) {
        const double skew = 1.0 + 0.02 * (tc.cfg.a_mn_major + tc.cfg.b_mn_major);
        // the vector epilogue wants the n index contiguous in C; anything else stores element-wise
        const double c_pen = g.c_s[5] == 1 ? 1.0 : (g.c_s[3] == 1 ? 1.3 : 1.6);
        // T of the node = the best over its implementation variants (tile width, CTA pair, cluster split-K)
        double best = kInf;
        // (a residual step's output and addend are residual-stream tensors, which a bf16 plan holds in fp32 unless told
        // otherwise: the epilogue's bytes, which the forms divide differently among their CTAs, are rated as such)
        if (n.res >= 0 && !p->opts.narrow_stream && g.dtype == FLUID_BF16) g.c_f32 = g.r_f32 = 1;
        // (a caller's op_variant request does not enter the rating: it swaps the variant of a step, not the plan)
        for (int code : gemm_tc_variants(p, g, 1)) {
          GemmTcHost tv;
          if (!gemm_tc_describe(g, &tv, code)) continue;
          best = std::min(best, gemm_tc_variant_cost(g, tv, 1));
        }
        if (best == kInf) best = fl / kTcPeak;
        return kLaunch + std::max(std::max(best, fl / (1.25 * kTcPeak)), by / kBw) * skew * c_pen;
      }
      const bool a_fast = g.a_s[5] == 1 || g.a_s[3] == 1, b_fast = g.b_s[5] == 1 || g.b_s[3] == 1,
                 c_fast = g.c_s[5] == 1 || g.c_s[3] == 1;
      const double pen = (a_fast ? 1.0 : 4.0) * (b_fast ? 1.0 : 4.0) * (c_fast ? 1.0 : 2.0);
      return kLaunch + std::max(fl / kSimtPeak, by / kBw) * pen;
    }
    case N_NORM: {
      const int rank = T[n.out].rank;
      if (perm_of(p, n.out, lo)[rank - 1] != rank - 1) return kInf;
      if (!same_perm(p, n.a, n.out, lo)) return kInf;
      if (n.res >= 0 && !same_perm(p, n.res, n.out, lo)) return kInf;
      return kLaunch + (2.0 + (n.res >= 0 ? 1.0 : 0.0)) * tbytes(p, n.out) / kBw;
    }
    case N_SOFTMAX: {
      const int rank = T[n.out].rank;
      const Perm& pm = perm_of(p, n.out, lo);
      if (pm[rank - 1] != rank - 1 || !same_perm(p, n.a, n.out, lo)) return kInf;
      if (n.sm_causal && pm[rank - 2] != rank - 2) return kInf;
      return kLaunch + (n.sm_causal ? 1.5 : 2.0) * tbytes(p, n.out) / kBw;
    }
    case N_ROPE:
      if (!same_perm(p, n.a, n.out, lo)) return kInf;
      return kLaunch + 2.0 * tbytes(p, n.out) / kBw;
    case N_ELTWISE: {
      if (!same_perm(p, n.a, n.out, lo)) return kInf;
      if (n.b >= 0 && !same_perm(p, n.b, n.out, lo)) return kInf;
      return kLaunch + (2.0 + (n.b >= 0 ? 1.0 : 0.0)) * tbytes(p, n.out) / kBw;
    }
    case N_TRANSPOSE: {
      if (transpose_is_alias(p, n, lo)) return 0.0;
      const TensorDesc &x = T[n.a], &y = T[n.out];
      const Perm &px = perm_of(p, n.a, lo), &py = perm_of(p, n.out, lo);
      const bool inner_kept = n.perm[py[y.rank - 1]] == px[x.rank - 1];
      return kLaunch + 2.0 * tbytes(p, n.out) / kBw * (inner_kept ? 1.0 : 1.25);
    }
    case N_SELECT:
      if (!is_identity(p, n.a, lo) || !is_identity(p, n.out, lo)) return kInf;
      return kLaunch + 2.0 * tbytes(p, n.out) / kBw;
    case N_ATTN_DECODE: {
      // q, k, v and the result are [B,1,heads,D] rows: any order of the leading dims, D contiguous
      for (int t : {n.a, n.b, n.v, n.out})
        if (perm_of(p, t, lo)[3] != 3) return kInf;
      if (!attn_decode_supported(T[n.out].dtype, (int)T[n.out].dims[3])) return kInf;
      return kLaunch + (tbytes(p, n.kc) + tbytes(p, n.vc)) / kBw;   // the whole cache: the row count is a run-time value
    }
    case N_ATTN: {
      AttnParams ap;
      AttnHost ah;
      if (!lower_attn(p, n, lo, &ap, &ah)) return kInf;
      double fl = 4.0 * ap.B * ap.NH * double(ap.S) * ap.S * ap.D;
      if (ap.causal) fl *= 0.5;
      const double by = tbytes(p, n.a) + tbytes(p, n.b) + tbytes(p, n.v) + tbytes(p, n.out);
      // K or V with the sequence index contiguous cost a little more (transposed operand path)
      return kLaunch + std::max(fl / (0.35 * kTcPeak), by / kBw) * (1.0 + 0.02 * (ap.k_mn_major + ap.v_k_major));
    }
  }
  return kInf;
}

// ---- evaluation wrapper: built-in table or the caller's eval() -----------------------------------
struct Evaluator {
  const fluid_plan_s* p;
  std::vector<int> lo;  // scratch: layout index per tensor
  double operator()(int node, const std::vector<int>& tids, const std::vector<int>& lidx) {
    const Node& n = p->nodes[node];
    if (p->opts.eval_variant) return best_variant(node, tids, lidx, nullptr);
    if (p->opts.eval) {
      return p->opts.eval(p->opts.eval_user, n.ops[0], (int)tids.size(), tids.data(), lidx.data());
    }
    for (size_t i = 0; i < tids.size(); ++i) lo[tids[i]] = lidx[i];
    return node_cost(p, n, lo.data());
  }
  // The caller's eval_variant over every variant of the node under these layouts: the minimum, and its arg-min.
  double best_variant(int node, const std::vector<int>& tids, const std::vector<int>& lidx, int* chosen) {
    const Node& n = p->nodes[node];
    for (size_t i = 0; i < tids.size(); ++i) lo[tids[i]] = lidx[i];
    std::vector<int> codes;
    GemmParams g;
    GemmTcHost tc;
    if (n.kind == N_GEMM && lower_gemm(p, n, lo.data(), &g) && gemm_tc_eligible(p, g, &tc)) codes = gemm_tc_variants(p, g, 1);
    if (codes.empty()) codes.push_back(0);
    double best = kInf;
    int arg = codes[0];
    for (int code : codes) {
      const double c = p->opts.eval_variant(p->opts.eval_user, n.ops[0], (int)tids.size(), tids.data(), lidx.data(), code);
      if (c < best) { best = c; arg = code; }
    }
    if (chosen) *chosen = arg;
    return best;
  }
  // Built-in table: the arg-min variant of a GEMM node under these layouts (0 if the node has none).
  int rated_variant(int node, const std::vector<int>& tids, const std::vector<int>& lidx) {
    const Node& n = p->nodes[node];
    for (size_t i = 0; i < tids.size(); ++i) lo[tids[i]] = lidx[i];
    GemmParams g;
    GemmTcHost tc;
    if (n.kind != N_GEMM || !lower_gemm(p, n, lo.data(), &g) || !gemm_tc_eligible(p, g, &tc)) return 0;
    if (n.res >= 0 && !p->opts.narrow_stream && g.dtype == FLUID_BF16) g.c_f32 = g.r_f32 = 1;   // as node_cost rates it
    double best = kInf;
    int arg = 0;
    for (int code : gemm_tc_variants(p, g, 1)) {
      GemmTcHost tv;
      if (!gemm_tc_describe(g, &tv, code)) continue;
      const double c = gemm_tc_variant_cost(g, tv, 1);
      if (c < best) { best = c; arg = code; }
    }
    return arg;
  }
};

static std::vector<int> node_tensors(const Node& n) {
  std::vector<int> v;
  auto add = [&](int t) {
    if (std::find(v.begin(), v.end(), t) == v.end()) v.push_back(t);
  };
  for (int t : n.ins) add(t);
  for (int t : n.outs) add(t);
  return v;
}

static double total_cost(fluid_plan_s* p, Evaluator& ev, const std::vector<int>& assign) {
  double c = 0;
  for (size_t i = 0; i < p->nodes.size(); ++i) {
    std::vector<int> tids = node_tensors(p->nodes[i]), l;
    for (int t : tids) l.push_back(assign[t]);
    c += ev((int)i, tids, l);
  }
  return c;
}

// ---- P1: graph -> linear sequence ------------------------------------------------------------------
static bool linearise(const fluid_graph_s& g, std::vector<int>* order) {
  const int n = (int)g.ops.size();
  std::vector<int> producer(g.tensors.size(), -1), indeg(n, 0);
  for (int o = 0; o < n; ++o)
    for (int t : g.ops[o].outs) producer[t] = o;
  std::vector<std::set<int>> pred(n);
  std::vector<std::vector<int>> succ(n);
  for (int o = 0; o < n; ++o)
    for (int t : g.ops[o].ins)
      if (producer[t] >= 0) pred[o].insert(producer[t]);
  for (int o = 0; o < n; ++o) {
    indeg[o] = (int)pred[o].size();
    for (int q : pred[o]) succ[q].push_back(o);
  }
  std::set<int> ready;
  for (int o = 0; o < n; ++o)
    if (indeg[o] == 0) ready.insert(o);
  order->clear();
  while (!ready.empty()) {
    int v = *ready.begin();
    ready.erase(ready.begin());
    order->push_back(v);
    for (int s : succ[v])
      if (--indeg[s] == 0) ready.insert(s);
  }
  return (int)order->size() == n;
}

// ---- fusion: graph ops -> planning nodes ----------------------------------------------------------
static void build_nodes(fluid_plan_s* p, const std::vector<int>& order) {
  const fluid_graph_s& g = p->graph;
  const int nops = (int)g.ops.size(), nt = (int)g.tensors.size();
  const bool fuse = p->opts.fusion != 0;
  std::vector<int> pos(nops), producer(nt, -1);
  std::vector<std::vector<int>> consumers(nt);
  for (int i = 0; i < nops; ++i) pos[order[i]] = i;
  for (int o = 0; o < nops; ++o) {
    for (int t : g.ops[o].outs) producer[t] = o;
    for (int t : g.ops[o].ins) consumers[t].push_back(o);
  }
  std::vector<char> absorbed(nops, 0);
  p->node_of_op.assign(nops, -1);
  p->folded.assign(nt, 0);
  auto sole_consumer = [&](int t) -> int {
    if (g.tensors[t].kind != FLUID_ACT || consumers[t].size() != 1) return -1;
    int c = consumers[t][0];
    return absorbed[c] ? -1 : c;
  };
  auto available_before = [&](int t, int at_pos) { return producer[t] < 0 || pos[producer[t]] < at_pos; };
  // the ROPE op producing tensor t, if it can run inside the CACHED_ATTENTION op `att` that consumes t as its query or
  // key: rotate-half pairing, position taken from the attention's own pos input, no other reader
  auto rope_into_decode = [&](int t, int att) -> int {
    const int r = producer[t];
    if (r < 0 || g.ops[r].kind != FLUID_OP_ROPE || g.tensors[t].kind != FLUID_ACT || consumers[t].size() != 1) return -1;
    const OpDesc& ro = g.ops[r];
    if (ro.attrs.rope_interleaved || ro.ins.size() != 2 || ro.ins[1] != g.ops[att].ins[5]) return -1;
    return r;
  };
  // ROPE ops that a later CACHED_ATTENTION takes over produce no node of their own
  if (fuse)
    for (int o = 0; o < nops; ++o) {
      if (g.ops[o].kind != FLUID_OP_CACHED_ATTENTION) continue;
      const int rq = rope_into_decode(g.ops[o].ins[0], o), rk = rope_into_decode(g.ops[o].ins[1], o);
      if (rq >= 0 && rk >= 0 && g.ops[rq].attrs.rope_base == g.ops[rk].attrs.rope_base) absorbed[rq] = absorbed[rk] = 1;
    }
  for (int oi = 0; oi < nops; ++oi) {
    const int o = order[oi];
    if (absorbed[o]) continue;
    const OpDesc& op = g.ops[o];
    Node n;
    n.ops.push_back(o);
    n.out = op.outs[0];
    n.a = op.ins[0];
    switch (op.kind) {
      case FLUID_OP_EMBED:
        n.kind = N_EMBED; n.b = op.ins[1]; n.pos = op.ins.size() > 2 ? op.ins[2] : -1;
        n.pos_off = op.ins.size() > 3 ? op.ins[3] : -1;
        break;
      case FLUID_OP_LINEAR:
      case FLUID_OP_BMM_QK:
      case FLUID_OP_BMM_PV: {
        n.kind = N_GEMM;
        n.b = op.ins[1];
        n.gemm_kind = op.kind == FLUID_OP_LINEAR ? G_LINEAR : (op.kind == FLUID_OP_BMM_QK ? G_QK : G_PV);
        n.contract = op.attrs.contract;
        n.scale = op.kind == FLUID_OP_BMM_QK ? op.attrs.scale : 1.0;
        if (op.kind == FLUID_OP_LINEAR && op.ins.size() > 2) n.bias = op.ins[2];
        if (fuse && op.kind == FLUID_OP_LINEAR) {
          int c = sole_consumer(n.out);
          if (c >= 0 && g.ops[c].kind == FLUID_OP_GELU) {
            n.act = g.ops[c].attrs.gelu_tanh ? ACT_GELU_TANH : ACT_GELU_ERF;
            absorbed[c] = 1; n.ops.push_back(c); p->folded[n.out] = 1; n.out = g.ops[c].outs[0];
            c = sole_consumer(n.out);
          }
          if (c >= 0 && g.ops[c].kind == FLUID_OP_ADD) {
            const int other = g.ops[c].ins[0] == n.out ? g.ops[c].ins[1] : g.ops[c].ins[0];
            if (other != n.out && available_before(other, oi)) {
              n.res = other;
              absorbed[c] = 1; n.ops.push_back(c); p->folded[n.out] = 1; n.out = g.ops[c].outs[0];
            }
          }
        }
        if (fuse && !p->opts.unfused_attention && op.kind == FLUID_OP_BMM_QK && g.tensors[n.out].dtype == FLUID_BF16 &&
            tc_kernel_available() && p->opts.gemm_path != 1 &&
            (g.tensors[n.a].dims[3] == 64 || g.tensors[n.a].dims[3] == 128)) {
          const int c1 = sole_consumer(n.out);
          if (c1 >= 0 && g.ops[c1].kind == FLUID_OP_SOFTMAX && (!g.ops[c1].attrs.causal ||
                                                                g.tensors[n.out].dims[2] == g.tensors[n.out].dims[3])) {
            const int sm_out = g.ops[c1].outs[0];
            const int c2 = sole_consumer(sm_out);
            if (c2 >= 0 && g.ops[c2].kind == FLUID_OP_BMM_PV && g.ops[c2].ins[0] == sm_out &&
                g.ops[c2].ins[1] != sm_out && available_before(g.ops[c2].ins[1], oi) && op.attrs.scale * g.ops[c1].attrs.scale > 0) {
              // only if the all-canonical layouts can be fed to the kernel (so that a plan always exists)
              Node trial = n;
              trial.kind = N_ATTN;
              trial.v = g.ops[c2].ins[1];
              trial.out = g.ops[c2].outs[0];
              trial.scale = op.attrs.scale * g.ops[c1].attrs.scale;
              trial.sm_causal = g.ops[c1].attrs.causal;
              std::vector<int> canon(nt, 0);
              AttnParams tap;
              AttnHost tah;
              if (!lower_attn(p, trial, canon.data(), &tap, &tah)) goto no_attention_fusion;
              n.kind = N_ATTN;
              n.v = g.ops[c2].ins[1];
              n.scale = op.attrs.scale * g.ops[c1].attrs.scale;
              n.sm_causal = g.ops[c1].attrs.causal;
              absorbed[c1] = absorbed[c2] = 1;
              n.ops.push_back(c1); n.ops.push_back(c2);
              p->folded[n.out] = 1; p->folded[sm_out] = 1;
              n.out = g.ops[c2].outs[0];
              break;
            }
          }
        }
      no_attention_fusion:
        if (fuse && op.kind == FLUID_OP_BMM_QK) {
          int c = sole_consumer(n.out);
          if (c >= 0 && g.ops[c].kind == FLUID_OP_SOFTMAX && g.ops[c].attrs.causal &&
              g.tensors[n.out].dims[2] == g.tensors[n.out].dims[3])
            n.causal = CAUSAL_SKIP_UPPER;
        }
        if (fuse && op.kind == FLUID_OP_BMM_PV) {
          int pr = producer[n.a];
          if (pr >= 0 && g.ops[pr].kind == FLUID_OP_SOFTMAX && g.ops[pr].attrs.causal &&
              g.tensors[n.a].dims[2] == g.tensors[n.a].dims[3])
            n.causal = CAUSAL_CLIP_K;
        }
        break;
      }
      case FLUID_OP_ADD:
      case FLUID_OP_MUL: {
        n.b = op.ins[1];
        int c = (fuse && op.kind == FLUID_OP_ADD) ? sole_consumer(n.out) : -1;
        if (c >= 0 && (g.ops[c].kind == FLUID_OP_LAYERNORM || g.ops[c].kind == FLUID_OP_RMSNORM) &&
            g.ops[c].ins[0] == n.out && available_before(g.ops[c].ins[1], oi) &&
            (g.ops[c].ins.size() < 3 || available_before(g.ops[c].ins[2], oi))) {
          n.kind = N_NORM;
          n.res = op.ins[1];
          n.rms = g.ops[c].kind == FLUID_OP_RMSNORM;
          n.eps = g.ops[c].attrs.eps;
          n.gamma = g.ops[c].ins[1];
          n.beta = n.rms ? -1 : g.ops[c].ins[2];
          absorbed[c] = 1; n.ops.push_back(c); p->folded[n.out] = 1; n.out = g.ops[c].outs[0];
          n.b = -1;
        } else {
          n.kind = N_ELTWISE;
          n.elt = op.kind == FLUID_OP_ADD ? ELT_ADD : ELT_MUL;
        }
        break;
      }
      case FLUID_OP_GELU:
        n.kind = N_ELTWISE; n.elt = op.attrs.gelu_tanh ? ELT_GELU_TANH : ELT_GELU_ERF;
        break;
      case FLUID_OP_SILU: {
        n.kind = N_ELTWISE; n.elt = ELT_SILU;
        int c = fuse ? sole_consumer(n.out) : -1;
        if (c >= 0 && g.ops[c].kind == FLUID_OP_MUL) {
          const int other = g.ops[c].ins[0] == n.out ? g.ops[c].ins[1] : g.ops[c].ins[0];
          if (other != n.out && available_before(other, oi)) {
            n.elt = ELT_SILU_MUL; n.b = other;
            absorbed[c] = 1; n.ops.push_back(c); p->folded[n.out] = 1; n.out = g.ops[c].outs[0];
          }
        }
        break;
      }
      case FLUID_OP_SOFTMAX:
        n.kind = N_SOFTMAX; n.sm_causal = op.attrs.causal; n.scale = op.attrs.scale;
        break;
      case FLUID_OP_LAYERNORM:
      case FLUID_OP_RMSNORM:
        n.kind = N_NORM; n.rms = op.kind == FLUID_OP_RMSNORM; n.eps = op.attrs.eps;
        n.gamma = op.ins[1]; n.beta = n.rms ? -1 : op.ins[2];
        break;
      case FLUID_OP_ROPE:
        n.kind = N_ROPE; n.rope_base = op.attrs.rope_base; n.rope_interleaved = op.attrs.rope_interleaved;
        n.pos = op.ins.size() > 1 ? op.ins[1] : -1;
        break;
      case FLUID_OP_CACHED_ATTENTION: {
        n.kind = N_ATTN_DECODE; n.b = op.ins[1]; n.v = op.ins[2]; n.kc = op.ins[3]; n.vc = op.ins[4]; n.pos = op.ins[5];
        n.scale = op.attrs.scale;
        // the rotary embedding of the query and the key at the same position, when both feed nothing else, runs
        // inside the attention step (the rotated tensors never exist)
        if (fuse) {
          const int rq = rope_into_decode(n.a, o), rk = rope_into_decode(n.b, o);
          if (rq >= 0 && rk >= 0 && g.ops[rq].attrs.rope_base == g.ops[rk].attrs.rope_base) {
            n.rope_fused = 1;
            n.rope_base = g.ops[rq].attrs.rope_base;
            p->folded[n.a] = p->folded[n.b] = 1;
            n.a = g.ops[rq].ins[0];
            n.b = g.ops[rk].ins[0];
            n.ops.push_back(rq); n.ops.push_back(rk);
          }
        }
        break;
      }
      case FLUID_OP_TRANSPOSE:
        n.kind = N_TRANSPOSE;
        for (int i = 0; i < 8; ++i) n.perm[i] = op.attrs.perm[i];
        break;
      case FLUID_OP_SELECT_LAST_TOKEN:
        n.kind = N_SELECT;
        break;
    }
    // distinct external inputs in role order
    auto add_in = [&](int t) {
      if (t >= 0 && std::find(n.ins.begin(), n.ins.end(), t) == n.ins.end()) n.ins.push_back(t);
    };
    if (n.ops.size() == 1) {
      for (int t : op.ins) add_in(t);
    } else {
      add_in(n.a); add_in(n.b); add_in(n.v); add_in(n.bias); add_in(n.res); add_in(n.gamma); add_in(n.beta); add_in(n.kc); add_in(n.vc); add_in(n.pos);
    }
    n.outs.push_back(n.out);
    for (int o2 : n.ops) p->node_of_op[o2] = (int)p->nodes.size();
    p->nodes.push_back(n);
  }
}

// ---- Algorithms 1 and 2 on the node graph -------------------------------------------------------------
struct NodeFlow {
  std::vector<std::vector<int>> pred, succ;  // node indices, pred sorted by anchor op id
  std::vector<int> anchor;                   // tie-break key: the node's first op id
};

static NodeFlow make_flow(const fluid_plan_s* p) {
  NodeFlow f;
  const int nn = (int)p->nodes.size();
  std::vector<int> producer(p->graph.tensors.size(), -1);
  f.pred.resize(nn);
  f.succ.resize(nn);
  f.anchor.resize(nn);
  for (int i = 0; i < nn; ++i) {
    f.anchor[i] = p->nodes[i].ops[0];
    for (int t : p->nodes[i].outs) producer[t] = i;
  }
  for (int i = 0; i < nn; ++i) {
    for (int t : p->nodes[i].ins) {
      int q = producer[t];
      if (q >= 0 && std::find(f.pred[i].begin(), f.pred[i].end(), q) == f.pred[i].end()) f.pred[i].push_back(q);
    }
    std::sort(f.pred[i].begin(), f.pred[i].end(), [&](int x, int y) { return f.anchor[x] < f.anchor[y]; });
    for (int q : f.pred[i]) f.succ[q].push_back(i);
  }
  return f;
}

// Algorithm 1: longest distances from the sub-flow's sources, then walk back from the farthest node.
static std::vector<int> find_longest_sequence(const NodeFlow& f, const std::vector<int>& nodes /*linear order*/,
                                              const std::vector<char>& inside) {
  std::map<int, int> dist, back;
  for (int v : nodes) {
    int best_d = -1, best_p = -1;
    for (int q : f.pred[v])
      if (inside[q] && dist[q] > best_d) {
        best_d = dist[q];
        best_p = q;
      }
    dist[v] = best_p >= 0 ? best_d + 1 : 0;
    back[v] = best_p;
  }
  int end = -1;
  for (int v : nodes)
    if (end < 0 || dist[v] > dist[end] || (dist[v] == dist[end] && f.anchor[v] < f.anchor[end])) end = v;
  std::vector<int> seq;
  for (int v = end; v >= 0; v = back[v]) seq.push_back(v);
  std::reverse(seq.begin(), seq.end());
  return seq;
}

// Algorithm 2: peel the longest sequence and recurse into each connected component of the rest.
static void split(const NodeFlow& f, std::vector<int> nodes, std::vector<std::vector<int>>* out) {
  if (nodes.empty()) return;
  const int nn = (int)f.pred.size();
  std::vector<char> inside(nn, 0);
  for (int v : nodes) inside[v] = 1;
  std::vector<int> seq = find_longest_sequence(f, nodes, inside);
  out->push_back(seq);
  for (int v : seq) inside[v] = 0;
  std::vector<int> rest;
  for (int v : nodes)
    if (inside[v]) rest.push_back(v);
  std::vector<int> by_anchor = rest;
  std::sort(by_anchor.begin(), by_anchor.end(), [&](int x, int y) { return f.anchor[x] < f.anchor[y]; });
  std::vector<char> seen(nn, 0);
  for (int start : by_anchor) {
    if (seen[start]) continue;
    std::vector<int> comp, stack{start};
    seen[start] = 1;
    while (!stack.empty()) {
      int v = stack.back();
      stack.pop_back();
      comp.push_back(v);
      for (int u : f.pred[v])
        if (inside[u] && !seen[u]) { seen[u] = 1; stack.push_back(u); }
      for (int u : f.succ[v])
        if (inside[u] && !seen[u]) { seen[u] = 1; stack.push_back(u); }
    }
    std::sort(comp.begin(), comp.end());  // node index order = linear order
    split(f, comp, out);
  }
}

// ---- Eq. 1 / Algorithm 3 ---------------------------------------------------------------------------------
struct Proposal { int tensor, layout; };

static bool dp_on_sequence(fluid_plan_s* p, Evaluator& ev, const std::vector<int>& seq,
                           const std::vector<int>& fixed /*per tensor, -1 = free*/, std::vector<Proposal>* props,
                           double* cost_out = nullptr) {
  const auto& T = p->graph.tensors;
  const int n = (int)seq.size();
  // chain edges e_0 .. e_n
  std::vector<int> edges(n + 1, -1);
  for (int t : p->nodes[seq[0]].ins)
    if (T[t].kind != FLUID_CONST) { edges[0] = t; break; }
  for (int i = 0; i + 1 < n; ++i) {
    int best = -1;
    for (int t : p->nodes[seq[i]].outs)
      for (int u : p->nodes[seq[i + 1]].ins)
        if (t == u && (best < 0 || t < best)) best = t;
    edges[i + 1] = best;
  }
  edges[n] = p->nodes[seq[n - 1]].outs[0];
  auto allowed = [&](int t) {
    std::vector<int> v;
    if (t < 0) { v.push_back(0); return v; }
    if (fixed[t] >= 0) { v.push_back(fixed[t]); return v; }
    for (int i = 0; i < (int)p->cands[t].size(); ++i) v.push_back(i);
    return v;
  };
  struct Back { int lp = -1; std::vector<int> side_assign; };
  std::vector<std::map<int, Back>> backs(n);
  std::vector<std::vector<int>> sides(n);
  std::map<int, double> prev;
  for (int l : allowed(edges[0])) prev[l] = 0.0;
  for (int i = 1; i <= n; ++i) {
    const int node = seq[i - 1], e_in = edges[i - 1], e_out = edges[i];
    std::vector<int> tids = node_tensors(p->nodes[node]);
    std::vector<int>& side = sides[i - 1];
    for (int t : tids)
      if (t != e_in && t != e_out) side.push_back(t);
    std::vector<std::vector<int>> side_opts;
    for (int s : side) side_opts.push_back(allowed(s));
    // argument order handed to eval: the node's tensors, inputs then outputs
    std::vector<int> lidx(tids.size(), 0);
    auto slot = [&](int t) { return int(std::find(tids.begin(), tids.end(), t) - tids.begin()); };
    std::map<int, double> cur;
    for (int l : allowed(e_out)) {
      double best = kInf;
      Back arg;
      for (int lp : allowed(e_in)) {
        if (std::isinf(prev[lp])) continue;
        std::vector<int> idx(side.size(), 0);
        while (true) {
          for (size_t s = 0; s < side.size(); ++s) lidx[slot(side[s])] = side_opts[s][idx[s]];
          if (e_in >= 0) lidx[slot(e_in)] = lp;
          lidx[slot(e_out)] = l;
          const double c = prev[lp] + ev(node, tids, lidx);
          if (c < best) {
            best = c;
            arg.lp = lp;
            arg.side_assign.clear();
            for (size_t s = 0; s < side.size(); ++s) arg.side_assign.push_back(side_opts[s][idx[s]]);
          }
          // next combination, last side tensor fastest
          int s = (int)side.size() - 1;
          while (s >= 0 && ++idx[s] == (int)side_opts[s].size()) idx[s--] = 0;
          if (s < 0) break;
        }
      }
      cur[l] = best;
      backs[i - 1][l] = arg;
    }
    prev = cur;
  }
  int l = -1;
  for (auto& kv : prev)
    if (l < 0 || kv.second < prev[l]) l = kv.first;
  if (cost_out) *cost_out = l < 0 ? kInf : prev[l];
  if (l < 0 || std::isinf(prev[l])) return false;
  props->push_back({edges[n], l});
  for (int i = n; i >= 1; --i) {
    const Back& b = backs[i - 1][l];
    for (size_t s = 0; s < sides[i - 1].size(); ++s) props->push_back({sides[i - 1][s], b.side_assign[s]});
    if (edges[i - 1] >= 0) props->push_back({edges[i - 1], b.lp});
    l = b.lp;
  }
  return true;
}

// ---- merge: majority vote, losers re-optimise ------------------------------------------------------------
static int plan_layouts(fluid_plan_s* p) {
  const int nt = (int)p->graph.tensors.size();
  Evaluator ev{p, std::vector<int>(nt, 0)};
  std::vector<int> canonical(nt, 0);
  p->canonical_cost = total_cost(p, ev, canonical);
  p->layout = canonical;
  p->cost = p->canonical_cost;
  NodeFlow flow = make_flow(p);
  std::vector<int> all(p->nodes.size());
  for (size_t i = 0; i < all.size(); ++i) all[i] = (int)i;
  p->sequences.clear();
  split(flow, all, &p->sequences);
  if (std::isinf(p->canonical_cost)) {
    set_error("the canonical layout assignment is not executable (an op has no kernel)");
    return FLUID_EUNSUPPORTED;
  }
  if (p->opts.force_canonical) return FLUID_OK;
  std::vector<int> fixed(nt, -1);
  std::vector<std::map<int, int>> votes;
  for (int round = 0; round <= nt + 1; ++round) {
    votes.assign(nt, {});
    for (const auto& seq : p->sequences) {
      std::vector<Proposal> props;
      if (!dp_on_sequence(p, ev, seq, fixed, &props)) {
        set_error("no supported layout assignment on a sequence");
        return FLUID_EUNSUPPORTED;
      }
      for (const Proposal& pr : props) votes[pr.tensor][pr.layout]++;
    }
    bool conflict = false;
    for (int t = 0; t < nt; ++t) {
      if (votes[t].size() <= 1) continue;
      conflict = true;
      int top = 0;
      for (auto& kv : votes[t]) top = std::max(top, kv.second);
      std::vector<int> tied;
      for (auto& kv : votes[t])
        if (kv.second == top) tied.push_back(kv.first);  // ascending layout index
      if (tied.size() == 1) {
        fixed[t] = tied[0];
        continue;
      }
      // a tie goes to the layout under which the re-optimised sequences cost least in total
      int best = -1;
      double best_cost = 0;
      for (int l : tied) {
        std::vector<int> trial = fixed;
        trial[t] = l;
        double c = 0;
        for (const auto& seq : p->sequences) {
          std::vector<Proposal> scratch;
          double sc = kInf;
          dp_on_sequence(p, ev, seq, trial, &scratch, &sc);
          c += sc;
        }
        if (best < 0 || c < best_cost) { best = l; best_cost = c; }
      }
      fixed[t] = best;
    }
    if (!conflict) break;
  }
  std::vector<int> assign(nt, 0);
  for (int t = 0; t < nt; ++t)
    if (!votes[t].empty()) assign[t] = votes[t].begin()->first;
  const double c = total_cost(p, ev, assign);
  if (c <= p->canonical_cost) {  // never worse than leaving every tensor canonical
    p->layout = assign;
    p->cost = c;
  }
  // the implementation variant each GEMM node was rated with under the final layouts is the one its step runs
  p->node_variant.assign(p->nodes.size(), 0);
  for (size_t i = 0; i < p->nodes.size(); ++i) {
    if (p->nodes[i].kind != N_GEMM) continue;
    std::vector<int> tids = node_tensors(p->nodes[i]), l;
    for (int t : tids) l.push_back(p->layout[t]);
    int code = 0;
    if (p->opts.eval_variant) ev.best_variant((int)i, tids, l, &code);
    else if (!p->opts.eval) code = ev.rated_variant((int)i, tids, l);
    p->node_variant[i] = code;
  }
  return FLUID_OK;
}

// ---- Algorithm 4: Greedy-by-Size --------------------------------------------------------------------------
static int64_t round_up(int64_t n, int64_t a) { return (n + a - 1) / a * a; }

// Algorithm 4 (Greedy-by-Size): records in the given order, each into a gap among the lifetime-overlapping records placed
// so far (first fit as printed, or the tightest gap as the prose has it), else at the tail.
static int64_t place_in_order(std::vector<ArenaRecord>& recs, const std::vector<int>& order, bool best_fit, bool no_reuse) {
  int64_t arena = FLUID_ARENA_HEADER;
  std::vector<int> placed;
  for (int ri : order) {
    ArenaRecord& r = recs[ri];
    std::vector<std::pair<int64_t, int64_t>> busy;
    for (int qi : placed) {
      const ArenaRecord& q = recs[qi];
      if (no_reuse || (q.first <= r.last && r.first <= q.last)) busy.push_back({q.offset, q.offset + q.bytes});
    }
    std::sort(busy.begin(), busy.end());
    int64_t cursor = FLUID_ARENA_HEADER, best_off = -1, best_gap = -1;
    for (auto& b : busy) {
      const int64_t gap = b.first - cursor;
      if (gap >= r.bytes) {
        if (!best_fit) {
          if (best_off < 0) { best_off = cursor; best_gap = gap; }
        } else if (best_off < 0 || gap < best_gap) {
          best_off = cursor; best_gap = gap;
        }
      }
      cursor = std::max(cursor, b.second);
    }
    r.offset = best_off >= 0 ? best_off : cursor;
    arena = std::max(arena, r.offset + r.bytes);
    placed.push_back(ri);
  }
  return arena;
}

// policy 0 / 1: the paper's order (size, descending) with first / best fit. policy 2 (not in the paper): the same
// placement run over a handful of orders and both fits, keeping the smallest arena; the paper's order comes first, so
// the result is never larger than policy 0's or 1's.
static void greedy_by_size(std::vector<ArenaRecord>& recs, int policy, bool no_reuse, size_t* arena_bytes) {
  std::vector<int> order(recs.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
  auto by_size = [&](int x, int y) {
    if (recs[x].bytes != recs[y].bytes) return recs[x].bytes > recs[y].bytes;
    if (recs[x].first != recs[y].first) return recs[x].first < recs[y].first;
    return recs[x].id < recs[y].id;
  };
  std::sort(order.begin(), order.end(), by_size);
  if (policy != 2) {
    *arena_bytes = (size_t)place_in_order(recs, order, policy == 1, no_reuse);
    return;
  }
  auto span = [&](int x) { return int64_t(recs[x].last - recs[x].first + 1); };
  std::vector<std::vector<int>> orders;
  orders.push_back(order);
  {  // long-lived records first, then size
    std::vector<int> o = order;
    std::stable_sort(o.begin(), o.end(), [&](int x, int y) { return span(x) > span(y); });
    orders.push_back(o);
  }
  {  // bytes x steps alive
    std::vector<int> o = order;
    std::stable_sort(o.begin(), o.end(), [&](int x, int y) { return recs[x].bytes * span(x) > recs[y].bytes * span(y); });
    orders.push_back(o);
  }
  {  // in order of first use
    std::vector<int> o = order;
    std::stable_sort(o.begin(), o.end(), [&](int x, int y) { return recs[x].first < recs[y].first; });
    orders.push_back(o);
  }
  {  // in reverse order of last use
    std::vector<int> o = order;
    std::stable_sort(o.begin(), o.end(), [&](int x, int y) { return recs[x].last > recs[y].last; });
    orders.push_back(o);
  }
  int64_t best = -1;
  std::vector<int64_t> best_off(recs.size(), 0);
  for (const auto& o : orders)
    for (int fit = 0; fit < 2; ++fit) {
      const int64_t a = place_in_order(recs, o, fit == 1, no_reuse);
      if (best < 0 || a < best) {
        best = a;
        for (size_t i = 0; i < recs.size(); ++i) best_off[i] = recs[i].offset;
      }
    }
  // Once more, for plans in which a few large records sit among many of one common size (a 43 MB SwiGLU product among
  // 16 MB projections): the large ones are placed as if they were a whole number of the common size, so the gaps they
  // leave hold whole records of that size, and alternately from the bottom and from the top of the space under the
  // largest live set, so that the common-size records around them can alternate too (a layer's scratch next to the
  // product below it in one layer, above it in the next). Offsets found for padded sizes are valid for the true ones;
  // the arena is measured with the true ones.
  if (!no_reuse && !recs.empty()) {
    std::vector<int64_t> sizes;
    for (const ArenaRecord& r : recs) sizes.push_back(r.bytes);
    std::sort(sizes.begin(), sizes.end());
    int64_t quantum = 0;
    int best_count = 0;
    for (size_t i = 0; i < sizes.size();) {
      size_t j = i;
      while (j < sizes.size() && sizes[j] == sizes[i]) ++j;
      if (int(j - i) > best_count || (int(j - i) == best_count && sizes[i] > quantum)) { best_count = int(j - i); quantum = sizes[i]; }
      i = j;
    }
    int last_step = 0;
    for (const ArenaRecord& r : recs) last_step = std::max(last_step, r.last);
    int64_t live = 0;   // largest live set, with the padded sizes
    std::vector<ArenaRecord> padded = recs;
    bool any = false;
    for (ArenaRecord& r : padded)
      if (quantum > 0 && r.bytes > quantum && r.bytes % quantum != 0) { r.bytes = (r.bytes + quantum - 1) / quantum * quantum; any = true; }
    for (int si = 0; si <= last_step; ++si) {
      int64_t sum = 0;
      for (const ArenaRecord& r : padded)
        if (r.first <= si && si <= r.last) sum += r.bytes;
      live = std::max(live, sum);
    }
    const int64_t ceiling = FLUID_ARENA_HEADER + live;
    if (any)
     for (const auto& ord : orders) {
      // a padded record takes the lowest gap or the highest place under the ceiling in turn, the others the lowest gap
      std::vector<int> placed;
      int turn = 0;
      for (int ri : ord) {
        ArenaRecord& r = padded[ri];
        std::vector<std::pair<int64_t, int64_t>> busy;
        for (int qi : placed) {
          const ArenaRecord& q = padded[qi];
          if (q.first <= r.last && r.first <= q.last) busy.push_back({q.offset, q.offset + q.bytes});
        }
        std::sort(busy.begin(), busy.end());
        const bool big = r.bytes != recs[ri].bytes;
        const bool from_top = big && (turn++ & 1);
        int64_t cursor = FLUID_ARENA_HEADER, low = -1, high = -1;
        for (auto& b : busy) {
          if (b.first - cursor >= r.bytes) {
            if (low < 0) low = cursor;
            if (b.first <= ceiling) high = b.first - r.bytes;
          }
          cursor = std::max(cursor, b.second);
        }
        if (low < 0) low = cursor;
        if (ceiling - cursor >= r.bytes) high = ceiling - r.bytes;
        r.offset = (from_top && high >= 0) ? high : low;
        placed.push_back(ri);
      }
      int64_t a = FLUID_ARENA_HEADER;
      for (size_t i = 0; i < recs.size(); ++i) a = std::max(a, padded[i].offset + recs[i].bytes);
      if (a < best) {
        best = a;
        for (size_t i = 0; i < recs.size(); ++i) best_off[i] = padded[i].offset;
      }
    }
  }
  for (size_t i = 0; i < recs.size(); ++i) recs[i].offset = best_off[i];
  *arena_bytes = (size_t)best;
}

// ---- lowering: nodes -> steps, aliases, lifetimes ----------------------------------------------------------
static int lower_and_place(fluid_plan_s* p) {
  const auto& T = p->graph.tensors;
  const int nt = (int)T.size();
  p->alias_root.resize(nt);
  for (int t = 0; t < nt; ++t) p->alias_root[t] = t;
  p->steps.clear();
  const int* lo = p->layout.data();
  Evaluator ev{p, std::vector<int>(nt, 0)};
  std::vector<char> taken(p->nodes.size(), 0);
  auto node_step_cost = [&](int ni) {
    std::vector<int> tids = node_tensors(p->nodes[ni]), l;
    for (int t : tids) l.push_back(lo[t]);
    return ev(ni, tids, l);
  };
  // sibling projections (same input, same shapes, no residual) can share one launch
  auto siblings_ok = [&](const Node& a, const Node& b) {
    if (b.kind != N_GEMM || b.gemm_kind != G_LINEAR || b.a != a.a || b.res >= 0 || b.act != a.act ||
        b.contract != a.contract || (a.bias >= 0) != (b.bias >= 0))
      return false;
    GemmParams ga, gb;
    GemmTcHost ta, tb;
    if (!lower_gemm(p, a, lo, &ga) || !lower_gemm(p, b, lo, &gb)) return false;
    if (!gemm_tc_eligible(p, ga, &ta) || !gemm_tc_eligible(p, gb, &tb)) return false;
    if (ga.M != gb.M || ga.N != gb.N || ga.K != gb.K || ga.N0 != gb.N0 || ga.M0 != gb.M0 || ga.K0 != gb.K0) return false;
    if (std::memcmp(&ta.cfg, &tb.cfg, sizeof(GemmTcCfg)) != 0) return false;
    for (int i = 0; i < 6; ++i)
      if (ga.a_s[i] != gb.a_s[i]) return false;
    for (int d = 0; d < 5; ++d)
      if (ta.b.dims[d] != tb.b.dims[d] || ta.b.strides[d] != tb.b.strides[d] || ta.b.box[d] != tb.b.box[d]) return false;
    return true;
  };
  for (int ni = 0; ni < (int)p->nodes.size(); ++ni) {
    if (taken[ni]) continue;
    const Node& n = p->nodes[ni];
    if (n.kind == N_TRANSPOSE && transpose_is_alias(p, n, lo)) {
      p->alias_root[n.out] = p->alias_root[n.a];
      continue;
    }
    Step s;
    s.node = ni;
    s.nodes.push_back(ni);
    s.cost = node_step_cost(ni);
    if (p->opts.fusion && n.kind == N_GEMM && n.gemm_kind == G_LINEAR && n.res < 0) {
      for (int nj = ni + 1; nj < (int)p->nodes.size() && s.nodes.size() < 3; ++nj) {
        if (taken[nj]) continue;
        const Node& m = p->nodes[nj];
        if (m.kind == N_GEMM && m.gemm_kind == G_LINEAR && m.a == n.a && siblings_ok(n, m)) {
          taken[nj] = 1;
          s.nodes.push_back(nj);
          s.cost += node_step_cost(nj) - kLaunch;
        }
      }
    }
    p->steps.push_back(s);
  }
  // SwiGLU: a grouped {gate, up} GEMM step followed by SiLU(gate) * up. When the pair qualifies for the CTA-pair
  // kernel, one CTA of each pair loads gate columns and the other up columns of the same 128 output columns, the
  // 256-wide accumulator holds both, and the epilogue writes SiLU(gate) * up: gate and up never reach memory.
  if (p->opts.fusion && p->opts.gemm_path == 0 && !p->opts.eval) {
    std::vector<int> n_uses(nt, 0);
    for (const Node& n : p->nodes)
      for (int t : n.ins) n_uses[t]++;
    for (int si = 0; si + 1 < (int)p->steps.size(); ++si) {
      Step& st = p->steps[si];
      if (st.nodes.size() != 2 || p->steps[si + 1].nodes.size() != 1) continue;
      const Node& e = p->nodes[p->steps[si + 1].node];
      if (e.kind != N_ELTWISE || e.elt != ELT_SILU_MUL) continue;
      int gi = -1, ui = -1;
      for (int k = 0; k < 2; ++k) {
        if (p->nodes[st.nodes[k]].out == e.a) gi = st.nodes[k];
        if (p->nodes[st.nodes[k]].out == e.b) ui = st.nodes[k];
      }
      if (gi < 0 || ui < 0 || gi == ui) continue;
      const Node &gn = p->nodes[gi], &un = p->nodes[ui];
      if (gn.kind != N_GEMM || un.kind != N_GEMM || gn.bias >= 0 || un.bias >= 0 || gn.res >= 0 || un.res >= 0 ||
          gn.act != ACT_NONE || un.act != ACT_NONE)
        continue;
      const int tg = gn.out, tu = un.out, to = e.out;
      if (n_uses[tg] != 1 || n_uses[tu] != 1 || T[tg].kind != FLUID_ACT || T[tu].kind != FLUID_ACT ||
          T[to].dtype != FLUID_BF16 || p->alias_root[tg] != tg || p->alias_root[tu] != tu)
        continue;
      if (lo[tg] != lo[tu] || lo[tg] != lo[to]) continue;   // the product takes the place (and strides) of gate
      GemmParams g;
      GemmTcHost tc;
      if (!lower_gemm(p, gn, lo, &g) || !gemm_tc_eligible(p, g, &tc)) continue;
      GemmParams gu;
      // a handful of rows: the weight-streaming kernel keeps the same tiles of gate and up in one CTA
      const bool rows = gemm_rows_eligible(g) && lower_gemm(p, un, lo, &gu) && gemm_rows_eligible(gu);
      GemmParams gpair[3] = {g, g, g};
      // (gemm_pair_eligible also answers no when the pair form is switched off in the environment)
      if (!rows && (!tc.cfg.pair || !gemm_pair_eligible(gpair, tc, 2) || g.batch != 1 || g.N % 128 != 0 || g.N0 % 128 != 0 ||
                    ((g.M + 127) / 128) % 2 != 0 || g.c_s[5] != 1))
        continue;
      st.nodes = {gi, ui, p->steps[si + 1].node};
      st.node = gi;
      st.swiglu = 1;
      st.cost += p->steps[si + 1].cost - kLaunch;
      p->folded[tg] = p->folded[tu] = 1;
      p->steps.erase(p->steps.begin() + si + 1);
    }
  }
  // Rotary embedding behind a grouped projection step (q, k, v): when the projections run as CTA pairs over 256-wide
  // tiles and the heads are 128 wide, each epilogue warp holds whole heads of its rows, so the rotation of q and k
  // runs in the epilogue and the unrotated tensors are never stored (nor rounded).
  if (p->opts.fusion && p->opts.gemm_path == 0 && !p->opts.eval && !p->opts.eval_variant) {
    std::vector<int> n_uses(nt, 0);
    for (const Node& n : p->nodes)
      for (int t : n.ins) n_uses[t]++;
    for (int si = 0; si < (int)p->steps.size(); ++si) {
      Step& st = p->steps[si];
      if (st.swiglu || st.norm_fused || st.nodes.size() < 2 || p->nodes[st.node].kind != N_GEMM) continue;
      const Node& n0 = p->nodes[st.node];
      GemmParams g;
      GemmTcHost tc;
      if (n0.bias >= 0 || n0.act != ACT_NONE || !lower_gemm(p, n0, lo, &g)) continue;
      if (!gemm_tc_eligible(p, g, &tc, gemm_variant_code(GV_PAIR, 256)) || !tc.cfg.pair) continue;
      GemmParams gs[3] = {g, g, g};
      if (!gemm_pair_eligible(gs, tc, (int)st.nodes.size()) || g.batch != 1 || g.N0 % 128 != 0 || g.N % 128 != 0 || g.c_s[5] != 1) continue;
      // the rotary steps that read this step's outputs, directly behind it
      std::vector<int> ropes;
      std::vector<int> order;   // GEMM nodes: rotated ones first (the launch applies the rotation per group)
      double base = 0;
      bool ok = true;
      for (int sj = si + 1; sj < (int)p->steps.size() && sj <= si + 2 && ok; ++sj) {
        const Step& sr = p->steps[sj];
        if (sr.nodes.size() != 1) break;
        const Node& r = p->nodes[sr.node];
        if (r.kind != N_ROPE) break;
        int owner = -1;
        for (int ni : st.nodes)
          if (p->nodes[ni].out == r.a) owner = ni;
        if (owner < 0 || r.rope_interleaved || r.pos >= 0 || n_uses[r.a] != 1 || T[r.a].kind != FLUID_ACT ||
            p->alias_root[r.a] != r.a || p->alias_root[r.out] != r.out || T[r.out].dtype != FLUID_BF16 || T[r.out].rank != 4 ||
            T[r.out].dims[3] != 128 || lo[r.a] != lo[r.out] || (base != 0 && base != r.rope_base))
          break;
        base = r.rope_base;
        ropes.push_back(sj);
        order.push_back(owner);
      }
      if (ropes.empty()) continue;
      (void)ok;
      for (int ni : st.nodes)
        if (std::find(order.begin(), order.end(), ni) == order.end()) order.push_back(ni);
      for (int sj : ropes) {
        const Node& r = p->nodes[p->steps[sj].node];
        st.cost += p->steps[sj].cost - kLaunch;
        p->folded[r.a] = 1;
      }
      const int first_rope = p->steps[ropes[0]].node, second_rope = ropes.size() > 1 ? p->steps[ropes[1]].node : -1;
      st.nodes = order;
      st.node = order[0];
      st.nodes.push_back(first_rope);
      if (second_rope >= 0) st.nodes.push_back(second_rope);
      st.rope_fused = (int)ropes.size();
      for (int k = (int)ropes.size() - 1; k >= 0; --k) p->steps.erase(p->steps.begin() + ropes[k]);
    }
  }
  // RMSNorm or LayerNorm in front of few-row GEMMs: when every reader of the normalised tensor is a GEMM of the next step and that
  // step runs the weight-streaming kernel, the normalisation runs inside it (the gain on the way in, 1/rms in the
  // epilogue) and the normalised tensor is never stored.
  if (p->opts.fusion && p->opts.gemm_path == 0 && !p->opts.eval && p->opts.split_k <= 0) {
    std::vector<int> n_uses(nt, 0);
    for (const Node& n : p->nodes)
      for (int t : n.ins) n_uses[t]++;
    for (int si = 0; si + 1 < (int)p->steps.size(); ++si) {
      const Step& sn = p->steps[si];
      if (sn.nodes.size() != 1) continue;
      const Node& nn = p->nodes[sn.node];
      if (nn.kind != N_NORM || nn.res >= 0 || T[nn.out].kind != FLUID_ACT || T[nn.out].dtype != FLUID_BF16 ||
          p->alias_root[nn.out] != nn.out || T[nn.gamma].kind != FLUID_CONST || lo[nn.gamma] != 0)
        continue;
      // LayerNorm: its bias rides along as one more activation row, so at most 15 rows, and not with SwiGLU
      const bool layer = !nn.rms;
      if (layer && (nn.beta < 0 || T[nn.beta].kind != FLUID_CONST || lo[nn.beta] != 0 || p->steps[si + 1].swiglu)) continue;
      Step& sg = p->steps[si + 1];
      int readers = 0;
      bool ok = true;
      for (int ni : sg.nodes) {
        const Node& m = p->nodes[ni];
        if (m.kind != N_GEMM) continue;   // the SiLU * up node of a SwiGLU step
        GemmParams g;
        ok = ok && m.a == nn.out && m.gemm_kind == G_LINEAR && lower_gemm(p, m, lo, &g) && gemm_rows_eligible(g);
        if (ok && layer) {   // room for the extra staged row
          GemmParams g1 = g;
          g1.M = g.M + 1;
          ok = g.M <= 15 && gemm_rows_eligible(g1);
        }
        ++readers;
      }
      if (!ok || readers == 0 || n_uses[nn.out] != readers) continue;
      sg.nodes.push_back(sn.node);
      sg.norm_fused = 1;
      sg.cost += sn.cost - kLaunch;
      p->folded[nn.out] = 1;
      p->steps.erase(p->steps.begin() + si);
    }
  }
  // RMS normalisation between two CTA-pair steps (pre-norm decoders at prefill sizes: o-proj / down -> RMSNorm ->
  // gate / up or q / k / v): the producer's residual epilogue holds whole 128-column slabs of the fp32 stream, so it also
  // writes bf16(x * gain) and the slabs' sums of squares, and the readers scale their accumulator rows by 1 / rms
  // ((x * gain / rms) . W = ((x * gain) . W) / rms): the normalisation's launch and its pass over the stream go.
  // bf16 is applied to x * gain instead of x * gain / rms: the same relative rounding.
  if (p->opts.fusion && p->opts.gemm_path == 0 && !p->opts.eval && !p->opts.eval_variant && !p->opts.narrow_stream &&
      p->opts.split_k <= 0 && !p->opts.no_norm_split) {
    std::vector<int> n_uses(nt, 0);
    for (const Node& n : p->nodes)
      for (int t : n.ins) n_uses[t]++;
    for (int si = 1; si + 1 < (int)p->steps.size(); ++si) {
      const Step& sn = p->steps[si];
      if (sn.nodes.size() != 1) continue;
      const Node& nn = p->nodes[sn.node];
      if (nn.kind != N_NORM || !nn.rms || nn.res >= 0 || T[nn.out].kind != FLUID_ACT || T[nn.out].dtype != FLUID_BF16 ||
          p->alias_root[nn.out] != nn.out || p->alias_root[nn.a] != nn.a || T[nn.gamma].kind != FLUID_CONST || lo[nn.gamma] != 0 ||
          !is_identity(p, nn.out, lo) || !is_identity(p, nn.a, lo) || T[nn.a].kind != FLUID_ACT || T[nn.a].dtype != FLUID_BF16)
        continue;
      Step& sp = p->steps[si - 1];
      Step& sc = p->steps[si + 1];
      if (sp.nodes.size() != 1 || sp.swiglu || sp.rope_fused || sp.norm_fused || sp.nrm_emit || sp.nrm_pre) continue;
      const Node& pn = p->nodes[sp.node];
      if (pn.kind != N_GEMM || pn.gemm_kind != G_LINEAR || pn.res < 0 || pn.out != nn.a || pn.act != ACT_NONE) continue;
      GemmParams g;
      GemmTcHost tc;
      if (!lower_gemm(p, pn, lo, &g) || !gemm_tc_eligible(p, g, &tc, gemm_variant_code(GV_PAIR, 256)) || !tc.cfg.pair) continue;
      GemmParams gs[3] = {g, g, g};
      bool like = true;
      for (int d = 0; d < 6; ++d) like = like && g.r_s[d] == g.c_s[d];
      if (!gemm_pair_eligible(gs, tc, 1) || !like || g.batch != 1 || g.N % 512 != 0 || g.N0 != g.N || g.M0 != g.M || g.c_s[5] != 1 ||
          g.c_s[3] != g.N || g.M % 256 != 0 || T[nn.out].numel() != (int64_t)g.M * g.N || T[nn.out].dims[T[nn.out].rank - 1] != g.N)
        continue;
      // the readers: every GEMM of the next step, which runs as CTA pairs with an epilogue that takes a row scale
      if (!(sc.swiglu || sc.rope_fused) || sc.nrm_pre || sc.norm_fused) continue;
      int readers = 0;
      bool ok = true;
      for (int ni : sc.nodes) {
        const Node& m = p->nodes[ni];
        if (m.kind != N_GEMM) continue;
        ok = ok && m.a == nn.out && m.gemm_kind == G_LINEAR;
        ++readers;
      }
      if (!ok || readers == 0 || n_uses[nn.out] != readers) continue;
      sp.nrm_emit = 1;
      sp.nrm_node = sn.node;
      sc.nrm_pre = 1;
      sc.nrm_node = sn.node;
      sc.nodes.push_back(sn.node);
      sc.cost += sn.cost - kLaunch;
      p->folded[nn.out] = 1;
      p->steps.erase(p->steps.begin() + si);
    }
  }
  // lifetimes in step indices, per alias group
  p->first_step.assign(nt, -1);
  p->last_step.assign(nt, -1);
  std::vector<int> gfirst(nt, -1), glast(nt, -1);
  for (int si = 0; si < (int)p->steps.size(); ++si) {
    for (int ni : p->steps[si].nodes) {
      const Node& n = p->nodes[ni];
      for (int t : n.outs) {
        int r = p->alias_root[t];
        if (gfirst[r] < 0) gfirst[r] = si;
        glast[r] = std::max(glast[r], si);
      }
      for (int t : n.ins) {
        int r = p->alias_root[t];
        if (gfirst[r] < 0) gfirst[r] = si;  // inputs and constants: alive from first use
        glast[r] = std::max(glast[r], si);
      }
    }
  }
  for (int t = 0; t < nt; ++t) {
    p->first_step[t] = gfirst[p->alias_root[t]];
    p->last_step[t] = glast[p->alias_root[t]];
  }
  // Residual-stream tensors of a bf16 graph are held in fp32: a tensor that feeds a
  // normalisation or a residual addition and is written by a kernel that can emit fp32. If a GEMM
  // also reads it as an operand, the producing norm writes a bf16 twin as well.
  p->wide.assign(nt, 0);
  std::vector<char> need_twin(nt, 0);
  if (!p->opts.narrow_stream) {
    std::vector<int> producer(nt, -1), group(nt, 0), stream_use(nt, 0), operand_use(nt, 0);
    for (int t = 0; t < nt; ++t) group[p->alias_root[t]]++;
    for (const Step& s : p->steps)
     for (int ni : s.nodes) {
      const Node& n = p->nodes[ni];
      producer[n.out] = (n.kind == N_ELTWISE && n.elt != ELT_ADD) ? -2 : n.kind;
      for (int t : n.ins) {
        const bool stream = (n.kind == N_NORM && (t == n.a || t == n.res)) || (n.kind == N_GEMM && t == n.res) ||
                            (n.kind == N_ELTWISE && n.elt == ELT_ADD);
        const bool also_operand = n.kind == N_GEMM && (t == n.a || t == n.b);
        if (stream) stream_use[t]++;
        if (!stream || also_operand) operand_use[t]++;
      }
    }
    for (int t = 0; t < nt; ++t) {
      if (T[t].dtype != FLUID_BF16 || T[t].kind != FLUID_ACT || p->folded[t] || group[t] != 1 || p->alias_root[t] != t)
        continue;
      const int pk = producer[t];
      const bool can = pk == N_NORM || pk == N_EMBED || pk == N_GEMM || pk == N_ELTWISE;
      if (!can || stream_use[t] == 0) continue;
      if (operand_use[t] > 0 && pk != N_NORM) continue;
      p->wide[t] = 1;
      need_twin[t] = operand_use[t] > 0;
    }
  }
  p->records.clear();
  p->record_of.assign(nt, -1);
  p->twin_record_of.assign(nt, -1);
  for (int t = 0; t < nt; ++t) {
    if (p->alias_root[t] != t || T[t].kind != FLUID_ACT || p->folded[t] || gfirst[t] < 0) continue;
    ArenaRecord r;
    r.root = t;
    r.id = t;
    const int64_t zone = p->opts.redzone_bytes > 0 ? round_up(p->opts.redzone_bytes, FLUID_SLOT_ALIGN) : 0;
    r.bytes = round_up(T[t].numel() * (p->wide[t] ? 4 : T[t].esize()), FLUID_SLOT_ALIGN) + zone;
    r.first = gfirst[t];
    r.last = glast[t];
    p->record_of[t] = (int)p->records.size();
    p->records.push_back(r);
    if (need_twin[t]) {
      ArenaRecord w = r;
      w.id = t + nt;
      w.twin = 1;
      w.bytes = round_up(T[t].numel() * T[t].esize(), FLUID_SLOT_ALIGN) + zone;
      p->twin_record_of[t] = (int)p->records.size();
      p->records.push_back(w);
    }
  }
  // In-place alias groups: a step whose every output element is written by the thread that read the same element of
  // one input (rotary embedding, element-wise ops, the residual operand of a GEMM epilogue) may write over that input
  // when this step is the input's last reader. Output and input then share one record whose lifetime is the union
  // of the two ("the most suitable slot" of the paper's memory-management paragraph is, for such a tensor, the one
  // its dying operand already holds). Same bytes, same storage dtype, same layout, no bf16 twin on either side.
  p->storage_root.assign(nt, -1);
  for (int t = 0; t < nt; ++t) p->storage_root[t] = p->alias_root[t];
  if (!p->opts.no_reuse && !p->opts.no_inplace) {
    std::vector<char> dead(p->records.size(), 0);
    auto find = [&](int r) {
      while (p->storage_root[r] != r) r = p->storage_root[r];
      return r;
    };
    for (int si = 0; si < (int)p->steps.size(); ++si) {
      const Step& st = p->steps[si];
      if (st.nodes.size() != 1) continue;
      const Node& n = p->nodes[st.node];
      int cand[2] = {-1, -1};
      if (n.kind == N_ROPE) cand[0] = n.a;
      else if (n.kind == N_GEMM && n.res >= 0) cand[0] = n.res;
      else if (n.kind == N_ELTWISE) { cand[0] = n.a; cand[1] = n.b; }
      else continue;
      const int rd = p->alias_root[n.out];
      if (rd != n.out || T[rd].kind != FLUID_ACT || p->record_of[rd] < 0 || p->twin_record_of[rd] >= 0) continue;
      for (int src : cand) {
        if (src < 0 || T[src].kind != FLUID_ACT) continue;
        const int ra = p->alias_root[src], rs = find(ra);
        if (rs == rd || p->record_of[rs] < 0 || p->twin_record_of[ra] >= 0 || p->twin_record_of[rs] >= 0) continue;
        ArenaRecord& a = p->records[p->record_of[rs]];
        ArenaRecord& d = p->records[p->record_of[rd]];
        if (a.bytes != d.bytes || p->wide[ra] != p->wide[rd] || a.last != si || d.first != si) continue;
        if (T[src].rank != T[n.out].rank || !same_perm(p, src, n.out, lo)) continue;
        bool same_dims = true;
        for (int i = 0; i < T[src].rank; ++i) same_dims = same_dims && T[src].dims[i] == T[n.out].dims[i];
        if (!same_dims) continue;
        a.last = d.last;
        dead[p->record_of[rd]] = 1;
        p->storage_root[rd] = rs;
        break;
      }
    }
    // drop the absorbed records, resolve every tensor to the record that holds it
    std::vector<int> remap(p->records.size(), -1);
    std::vector<ArenaRecord> kept;
    for (size_t i = 0; i < p->records.size(); ++i)
      if (!dead[i]) { remap[i] = (int)kept.size(); kept.push_back(p->records[i]); }
    p->records.swap(kept);
    for (int t = 0; t < nt; ++t) {
      if (p->record_of[t] >= 0) p->record_of[t] = remap[p->record_of[t]];
      if (p->twin_record_of[t] >= 0) p->twin_record_of[t] = remap[p->twin_record_of[t]];
    }
    for (int t = 0; t < nt; ++t) p->storage_root[t] = find(p->alias_root[t]);
    for (int t = 0; t < nt; ++t)
      if (p->storage_root[t] != p->alias_root[t]) p->record_of[p->alias_root[t]] = p->record_of[p->storage_root[t]];
  }
  // per-step scratch: split-K partial tiles of GEMM steps with too few output tiles to fill the GPU
  for (int si = 0; si < (int)p->steps.size(); ++si) {
    Step& st = p->steps[si];
    const Node& n0 = p->nodes[st.node];
    if (n0.kind != N_GEMM || p->opts.split_k <= 0) continue;
    GemmParams g;
    GemmTcHost tc;
    if (!lower_gemm(p, n0, lo, &g) || !gemm_tc_eligible(p, g, &tc)) continue;
    g.c_f32 = p->wide[n0.out];
    g.r_f32 = n0.res >= 0 ? p->wide[n0.res] : 0;
    bool same_width = true;
    for (int nj : st.nodes) same_width = same_width && p->wide[p->nodes[nj].out] == p->wide[n0.out];
    if (!same_width) continue;
    int64_t bytes = 0;
    st.split_k = gemm_split_k(g, tc, (int)st.nodes.size(), &bytes);
    if (st.split_k <= 1) continue;
    ArenaRecord r;
    r.root = -1;
    r.step = si;
    r.id = 2 * nt + si;
    r.bytes = round_up(bytes, FLUID_SLOT_ALIGN);
    r.first = r.last = si;
    st.scratch_bytes = r.bytes;
    st.scratch_record = (int)p->records.size();
    p->records.push_back(r);
  }
  // scratch of a split RMS normalisation: bf16(x * gain) and the slabs' sums of squares, from the step that writes
  // them to the step that reads them (the next one)
  for (int si = 0; si + 1 < (int)p->steps.size(); ++si) {
    Step& st = p->steps[si];
    if (!st.nrm_emit) continue;
    const Node& nn = p->nodes[st.nrm_node];
    const int64_t n = T[nn.out].dims[T[nn.out].rank - 1], m = T[nn.out].numel() / n;
    // (two slices: the first has exactly the size the normalised tensor's own slice would have had)
    ArenaRecord r;
    r.root = -1;
    r.step = si;
    r.id = 3 * nt + si;
    r.bytes = round_up(m * n * 2, FLUID_SLOT_ALIGN);
    r.first = si;
    r.last = si + 1;
    st.nrm_record = p->steps[si + 1].nrm_record = (int)p->records.size();
    p->records.push_back(r);
    r.id = 3 * nt + (int)p->steps.size() + si;
    r.bytes = round_up(m * (n / 128) * 4, FLUID_SLOT_ALIGN);
    st.nrm_ss_record = p->steps[si + 1].nrm_ss_record = (int)p->records.size();
    p->records.push_back(r);
  }
  greedy_by_size(p->records, p->opts.arena_policy, p->opts.no_reuse != 0, &p->arena_bytes);
  // reference figures: one slice per tensor, and the largest live set
  int64_t naive = FLUID_ARENA_HEADER, live = 0;
  for (const ArenaRecord& r : p->records) naive += r.bytes;
  for (int si = 0; si < (int)p->steps.size(); ++si) {
    int64_t s = 0;
    for (const ArenaRecord& r : p->records)
      if (r.first <= si && si <= r.last) s += r.bytes;
    live = std::max(live, s);
  }
  p->naive_bytes = (size_t)naive;
  p->live_bound = (size_t)(live + FLUID_ARENA_HEADER);
  return finalize_steps(p);
}

}  // namespace fluid

using namespace fluid;

extern "C" {

void fluid_plan_default_options(fluid_plan_options* o) {
  if (!o) return;
  std::memset(o, 0, sizeof(*o));
  o->fusion = 1;
}

int fluid_plan(const fluid_graph_t* g, const fluid_layout_candidates* cands, const fluid_plan_options* opts,
               fluid_plan_t** out) {
  if (!g || !out) {
    set_error("null argument");
    return FLUID_EINVAL;
  }
  *out = nullptr;
  if (g->ops.empty()) {
    set_error("empty graph");
    return FLUID_EINVAL;
  }
  fluid_plan_s* p = new (std::nothrow) fluid_plan_s();
  if (!p) {
    set_error("out of host memory");
    return FLUID_ENOMEM;
  }
  p->graph = *g;
  if (opts) p->opts = *opts;
  else fluid_plan_default_options(&p->opts);
  if (p->opts.eval || p->opts.eval_variant) p->opts.fusion = 0;
  if (p->opts.op_variant && p->opts.n_op_variant > 0) p->op_variant.assign(p->opts.op_variant, p->opts.op_variant + p->opts.n_op_variant);
  p->opts.op_variant = nullptr;   // the caller's array is not kept
  p->opts.n_op_variant = 0;
  const int nt = (int)g->tensors.size();
  // layout candidates
  p->cands.assign(nt, {});
  if (cands && cands->n_tensors != nt) {
    set_error("layout_candidates covers %d tensors, graph has %d", cands->n_tensors, nt);
    delete p;
    return FLUID_EINVAL;
  }
  size_t cursor = 0;
  for (int t = 0; t < nt; ++t) {
    const TensorDesc& td = g->tensors[t];
    const int nc = cands ? cands->n_cands[t] : 0;
    if (nc < 0 || nc > 64) {
      set_error("tensor %d: bad candidate count %d", t, nc);
      delete p;
      return FLUID_EINVAL;
    }
    for (int c = 0; c < nc; ++c) {
      Perm pm = identity_perm();
      int seen = 0;
      bool ok = true;
      for (int i = 0; i < td.rank; ++i) {
        int v = cands->perms[cursor + i];
        ok = ok && v >= 0 && v < td.rank && !(seen & (1 << v));
        if (ok) { seen |= 1 << v; pm[i] = (int8_t)v; }
      }
      cursor += td.rank;
      if (ok && c == 0)
        for (int i = 0; i < td.rank; ++i) ok = ok && pm[i] == i;
      if (!ok) {
        set_error("tensor %d: candidate %d is not a permutation (or the first is not the identity)", t, c);
        delete p;
        return FLUID_EINVAL;
      }
      // the caller's buffers stay canonical whatever the list says
      if ((td.kind == FLUID_INPUT || td.kind == FLUID_OUTPUT || td.kind == FLUID_STATE) && c > 0) continue;
      p->cands[t].push_back(pm);
    }
    if (p->cands[t].empty()) p->cands[t].push_back(identity_perm());
  }
  // inputs / outputs in declaration order
  p->input_slot.assign(nt, -1);
  p->output_slot.assign(nt, -1);
  p->const_ptr.assign(nt, nullptr);
  int ni = 0, no = 0;
  for (int t = 0; t < nt; ++t) {
    if (g->tensors[t].kind == FLUID_INPUT || g->tensors[t].kind == FLUID_STATE) p->input_slot[t] = ni++;
    if (g->tensors[t].kind == FLUID_OUTPUT) p->output_slot[t] = no++;
  }
  std::vector<int> order;
  if (!linearise(p->graph, &order)) {
    set_error("graph has a cycle");
    delete p;
    return FLUID_EINVAL;
  }
  build_nodes(p, order);
  int rc = plan_layouts(p);
  if (rc == FLUID_OK) rc = lower_and_place(p);
  if (rc != FLUID_OK) {
    delete p;
    return rc;
  }
  *out = p;
  return FLUID_OK;
}

void fluid_plan_destroy(fluid_plan_t* p) { delete p; }

size_t fluid_plan_arena_bytes(const fluid_plan_t* p) { return p ? p->arena_bytes : 0; }
size_t fluid_plan_arena_naive_bytes(const fluid_plan_t* p) { return p ? p->naive_bytes : 0; }
size_t fluid_plan_arena_live_bound_bytes(const fluid_plan_t* p) { return p ? p->live_bound : 0; }
double fluid_plan_cost(const fluid_plan_t* p) { return p ? p->cost : 0.0; }
double fluid_plan_canonical_cost(const fluid_plan_t* p) { return p ? p->canonical_cost : 0.0; }

int fluid_plan_tensor_info(const fluid_plan_t* p, int t, int* layout_index, int* perm, int64_t* offset,
                           int64_t* bytes, int* first_step, int* last_step, int* alias_of) {
  if (!p || t < 0 || t >= (int)p->graph.tensors.size()) {
    set_error("bad plan or tensor id");
    return FLUID_EINVAL;
  }
  const TensorDesc& td = p->graph.tensors[t];
  if (layout_index) *layout_index = p->layout[t];
  if (perm)
    for (int i = 0; i < td.rank; ++i) perm[i] = p->cands[t][p->layout[t]][i];
  const int root = p->storage_root.empty() ? p->alias_root[t] : p->storage_root[t];   // the tensor whose record holds this one (a view or an in-place result)
  const int rec = p->record_of[root];
  if (offset) *offset = rec >= 0 ? p->records[rec].offset : -1;
  if (bytes) *bytes = rec >= 0 ? p->records[rec].bytes : td.numel() * td.esize();
  if (first_step) *first_step = p->first_step[t];
  if (last_step) *last_step = p->last_step[t];
  if (alias_of) *alias_of = root;
  return FLUID_OK;
}

int fluid_plan_num_records(const fluid_plan_t* p) { return p ? (int)p->records.size() : 0; }

int fluid_plan_record_info(const fluid_plan_t* p, int index, int* record_id, int* tensor_id, int* is_twin,
                           int* storage_dtype, int64_t* offset, int64_t* bytes, int* first_step, int* last_step) {
  if (!p || index < 0 || index >= (int)p->records.size()) {
    set_error("bad plan or record index");
    return FLUID_EINVAL;
  }
  const ArenaRecord& r = p->records[index];
  if (record_id) *record_id = r.id;
  if (tensor_id) *tensor_id = r.root;
  if (is_twin) *is_twin = r.twin;
  if (storage_dtype) *storage_dtype = r.root < 0 ? FLUID_F32 : ((p->wide[r.root] && !r.twin) ? FLUID_F32 : p->graph.tensors[r.root].dtype);
  if (offset) *offset = r.offset;
  if (bytes) *bytes = r.bytes;
  if (first_step) *first_step = r.first;
  if (last_step) *last_step = r.last;
  return FLUID_OK;
}

int fluid_plan_num_steps(const fluid_plan_t* p) { return p ? (int)p->steps.size() : 0; }

int fluid_plan_gemm_variants(const fluid_plan_t* p, int op_id, int* codes, int capacity, int* n_out, int* chosen) {
  if (!p || !n_out || op_id < 0 || op_id >= (int)p->node_of_op.size()) {
    set_error("gemm variants: bad plan or op id");
    return FLUID_EINVAL;
  }
  *n_out = 0;
  if (chosen) *chosen = 0;
  const int ni = p->node_of_op[op_id];
  if (ni < 0 || p->nodes[ni].kind != N_GEMM || p->nodes[ni].ops[0] != op_id) return FLUID_OK;
  // the step this node anchors (a grouped sibling launch is listed under its first node)
  for (const Step& s : p->steps) {
    if (s.kernel != FLUID_K_GEMM_TC || s.nodes.empty() || s.nodes[0] != ni) continue;
    const int n_group = s.swiglu ? 2 : std::max<int>(1, (s.variant >> 20) & 15);
    const std::vector<int> v = gemm_tc_variants(p, s.gemm, n_group);
    *n_out = (int)v.size();
    for (int i = 0; i < (int)v.size() && codes && i < capacity; ++i) codes[i] = v[i];
    if (chosen) {
      const int form = ((s.variant >> 28) & 1) ? GV_CLUSTER : (((s.variant >> 29) & 1) ? GV_PAIR : GV_SINGLE);
      *chosen = gemm_variant_code(form, (s.variant >> 8) & 0xfff);
    }
    return FLUID_OK;
  }
  return FLUID_OK;
}

int fluid_plan_step_info(const fluid_plan_t* p, int step, fluid_step_info* info) {
  if (!p || !info || step < 0 || step >= (int)p->steps.size()) {
    set_error("bad plan or step index");
    return FLUID_EINVAL;
  }
  const Step& s = p->steps[step];
  std::memset(info, 0, sizeof(*info));
  info->kernel = s.kernel;
  info->variant = s.variant;
  // (a normalisation whose second half this step runs is listed first: its result is what the step's GEMMs read)
  std::vector<int> order(s.nodes.begin(), s.nodes.end());
  if (s.nrm_pre && !order.empty()) std::rotate(order.begin(), order.end() - 1, order.end());
  for (int ni : order) {
    const Node& n = p->nodes[ni];
    for (int o : n.ops)
      if (info->n_ops < 8) info->ops[info->n_ops++] = o;
    // (tensors that a fused step keeps to itself are neither read from nor written to memory)
    for (int t : n.ins) {
      bool seen = p->folded[t] != 0;
      for (int i = 0; i < info->n_in; ++i) seen = seen || info->in_ids[i] == t;
      if (!seen && info->n_in < 8) info->in_ids[info->n_in++] = t;
    }
    for (int t : n.outs)
      if (!p->folded[t] && info->n_out < 4) info->out_ids[info->n_out++] = t;
  }
  info->cost = s.cost;
  info->flops = s.flops;
  info->bytes = s.bytes;
  return FLUID_OK;
}

int fluid_plan_num_sequences(const fluid_plan_t* p) { return p ? (int)p->sequences.size() : 0; }

int fluid_plan_sequence(const fluid_plan_t* p, int index, int* node_ids, int capacity, int* length) {
  if (!p || index < 0 || index >= (int)p->sequences.size() || !length) {
    set_error("bad plan or sequence index");
    return FLUID_EINVAL;
  }
  const auto& s = p->sequences[index];
  *length = (int)s.size();
  if (node_ids)
    for (int i = 0; i < (int)s.size() && i < capacity; ++i) node_ids[i] = p->nodes[s[i]].ops[0];
  return FLUID_OK;
}

int fluid_plan_bind_constant(fluid_plan_t* p, int t, const void* dev_ptr) {
  if (!p || t < 0 || t >= (int)p->graph.tensors.size() || p->graph.tensors[t].kind != FLUID_CONST) {
    set_error("bind_constant: not a constant tensor");
    return FLUID_EINVAL;
  }
  if (!dev_ptr || (reinterpret_cast<uintptr_t>(dev_ptr) & 15)) {
    set_error("bind_constant: pointer must be non-null and 16-byte aligned");
    return FLUID_EALIGN;
  }
  std::lock_guard<std::mutex> lk(p->mu);
  p->const_ptr[t] = dev_ptr;
  p->maps_valid = false;
  return FLUID_OK;
}

}  // extern "C"
