// fluid_run(): the arena executor. Walks the plan's step list, binds every tensor to
// arena_ptr + offset (or to a bound constant / caller buffer) and launches one kernel per step on
// the caller's stream. No allocation, no synchronisation, no copies (the paper's "user only
// needs to allocate a big block of buffer", Sec. "Evaluation", memory-allocation paragraph).
#include <cmath>
#include <atomic>
#include <cstdio>
#include <vector>

#include "fluid_internal.h"

namespace fluid {

static std::atomic<int64_t> g_launches{0};

static void perm_strides(const fluid_plan_s* p, int t, int64_t* st) {
  strides_of(p->graph.tensors[t], p->cands[t][p->layout[t]], st);
}

// Derive every step's launch payload from the final layouts (host only, no device access).
int finalize_steps(fluid_plan_s* p) {
  const auto& T = p->graph.tensors;
  const int* lo = p->layout.data();
  for (Step& s : p->steps) {
    const Node& n = p->nodes[s.node];
    const TensorDesc& ty = T[n.out];
    const double es = (double)ty.esize();
    // A caller's cost function may rate a combination of layouts the kernels cannot run (the built-in table
    // never does): refuse it here, at plan time, rather than run a kernel on strides it does not understand.
    // (Such a plan is kept: its sequences, layouts and arena can still be inspected. It refuses to run.)
    bool feasible = true;
    for (int ni : s.nodes) {
      if (!std::isfinite(node_cost(p, p->nodes[ni], lo))) {
        if (!p->opts.eval && !p->opts.eval_variant) {
          set_error("step for op %d: no kernel runs this operator with the chosen layouts", p->nodes[ni].ops[0]);
          return FLUID_EUNSUPPORTED;
        }
        if (p->not_runnable_op < 0) p->not_runnable_op = p->nodes[ni].ops[0];
        feasible = false;
      }
    }
    if (!feasible) continue;
    switch (n.kind) {
      case N_EMBED: {
        s.kernel = FLUID_K_EMBED;
        EmbedParams e{};
        e.dtype = ty.dtype;
        e.tokens = int(ty.dims[0] * ty.dims[1]);
        e.S = (int)ty.dims[1];
        e.H = (int)ty.dims[2];
        e.V = (int)T[n.b].dims[0];
        e.y_f32 = p->wide[n.out];
        e.P = n.pos >= 0 ? (int)T[n.pos].dims[0] : 0;
        e.pos_off_stride = (n.pos_off >= 0 && T[n.pos_off].dims[0] > 1) ? 1 : 0;
        s.embed = e;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.b; s.t_ptr[2] = n.pos; s.t_ptr[3] = n.out; s.t_ptr[4] = n.pos_off;
        s.bytes = es * ty.numel() * (n.pos >= 0 ? 3.0 : 2.0) + 4.0 * e.tokens;
        break;
      }
      case N_GEMM: {
        if (!lower_gemm(p, n, lo, &s.gemm)) {
          set_error("step for op %d: GEMM cannot be lowered under the chosen layouts", n.ops[0]);
          return FLUID_EUNSUPPORTED;
        }
        const GemmParams& g = s.gemm;
        // the variant the planner rated best for this node (or the caller asked for); the fused SwiGLU form exists for CTA pairs only
        int gv = (s.swiglu || s.rope_fused || s.nrm_emit) ? gemm_variant_code(GV_PAIR, 256) : gemm_variant_of(p, n);
        // A node is rated on its own; siblings that share a launch multiply the tiles, which moves the wave count the
        // rating turns on: the group is rated again as a group (unless the caller named a variant or rates them itself).
        const int n_sib = (s.swiglu || s.rope_fused || s.nrm_emit) ? 1 : int(s.nodes.size()) - s.norm_fused - s.nrm_pre;
        const int anchor = n.ops.empty() ? -1 : n.ops[0];
        const bool asked = anchor >= 0 && anchor < (int)p->op_variant.size() && p->op_variant[anchor] != 0;
        if (n_sib > 1 && !asked && !p->opts.eval_variant) {
          double best = kInf;
          for (int code : gemm_tc_variants(p, g, n_sib)) {
            GemmTcHost tv;
            if (!gemm_tc_describe(g, &tv, code)) continue;
            const double c = gemm_tc_variant_cost(g, tv, n_sib);
            if (c < best) { best = c; gv = code; }
          }
        }
        s.kernel = gemm_tc_eligible(p, g, &s.tc, gv) ? FLUID_K_GEMM_TC : FLUID_K_GEMM_SIMT;
        if (s.kernel == FLUID_K_GEMM_TC)
          s.variant = (s.tc.cfg.a_mn_major ? 1 : 0) | (s.tc.cfg.b_mn_major ? 2 : 0) | (s.tc.cfg.bn << 8);
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.b; s.t_ptr[2] = n.out; s.t_ptr[3] = n.bias; s.t_ptr[4] = n.res;
        s.t_narrow[0] = s.t_narrow[1] = 1;
        s.gemm.c_f32 = p->wide[n.out];
        s.gemm.r_f32 = n.res >= 0 ? p->wide[n.res] : 0;
        s.gemm.b_const = p->graph.tensors[n.b].kind == FLUID_CONST ? 1 : 0;
        double fl = 2.0 * double(g.batch) * g.M * double(g.N) * g.K;
        double a = double(g.batch) * g.M * double(g.K), b = double(g.batch) * g.K * double(g.N),
               c = double(g.batch) * g.M * double(g.N);
        if (g.causal != CAUSAL_NONE) {
          const double tri = 0.5 * (1.0 + 1.0 / g.M);
          fl *= tri;
          if (g.causal == CAUSAL_SKIP_UPPER) c *= tri;
          else a *= tri;
        }
        s.flops = fl;
        s.bytes = es * (a + b + (g.has_bias ? g.N : 0)) + c * (s.gemm.c_f32 ? 4.0 : es) + (g.has_res ? c * (s.gemm.r_f32 ? 4.0 : es) : 0.0);
        // split RMS normalisation: bf16(x * gain) and the slabs' sums of squares, written by one side, read by the other
        if (s.nrm_emit) s.bytes += es * c + 4.0 * g.M * (g.N / 128);
        if (s.nrm_pre) s.bytes += 4.0 * g.M * (g.K / 128);
        // SwiGLU step: the only tensor written is the product, which takes gate's place
        const size_t n_gemm = s.swiglu ? 2 : s.nodes.size() - s.norm_fused - s.rope_fused - s.nrm_pre;
        if (s.swiglu) {
          s.t_ptr[2] = p->nodes[s.nodes[2]].out;
          s.gemm.c_f32 = 0;
          s.bytes = es * (a + 2.0 * b + c);
          s.flops = 2.0 * fl;
        }
        // grouped siblings: same A, own B / C / bias
        for (size_t gi = 1; gi < n_gemm; ++gi) {
          const Node& m = p->nodes[s.nodes[gi]];
          GemmParams& gx = s.gemm_x[gi - 1];
          if (!lower_gemm(p, m, lo, &gx) || !gemm_tc_eligible(p, gx, &s.tc_x[gi - 1], gv) || s.kernel != FLUID_K_GEMM_TC ||
              s.tc_x[gi - 1].cfg.bn != s.tc.cfg.bn || s.tc_x[gi - 1].cfg.pair != s.tc.cfg.pair) {
            set_error("step for op %d: sibling GEMM cannot share a launch", m.ops[0]);
            return FLUID_EUNSUPPORTED;
          }
          gx.c_f32 = p->wide[m.out];
          gx.b_const = p->graph.tensors[m.b].kind == FLUID_CONST ? 1 : 0;
          s.x_ptr[gi - 1][0] = m.b; s.x_ptr[gi - 1][1] = s.swiglu ? -1 : m.out; s.x_ptr[gi - 1][2] = m.bias;
          if (s.swiglu) continue;
          s.flops += fl;
          s.bytes += es * (b + c + (g.has_bias ? g.N : 0));
        }
        if (n_gemm > 1) s.variant |= int(n_gemm) << 20;
        // fused rotary embeddings: the first rope_fused projections write their rotated result (the rope nodes' outputs)
        for (int ri = 0; ri < s.rope_fused; ++ri) {
          const Node& rn = p->nodes[s.nodes[n_gemm + ri]];
          GemmParams& gr = ri == 0 ? s.gemm : s.gemm_x[ri - 1];
          gr.rope = 1;
          gr.rope_S = (int)T[rn.out].dims[1];
          if (ri == 0) s.t_ptr[2] = rn.out; else s.x_ptr[ri - 1][1] = rn.out;
          rope_freq_fill(s.rope_freq, rn.rope_base, (int)T[rn.out].dims[3]);
          s.bytes -= 0.0;
        }
        if (s.rope_fused) s.variant |= 1 << 30;
        // a handful of rows: the weight-streaming kernel, when every GEMM of the step has k contiguous on both sides
        if (p->opts.gemm_path == 0 && s.split_k <= 1 && g.dtype == FLUID_BF16) {
          bool rows = gemm_rows_eligible(s.gemm);
          for (size_t gi = 1; gi < n_gemm; ++gi) rows = rows && gemm_rows_eligible(s.gemm_x[gi - 1]);
          if (rows) {
            s.kernel = FLUID_K_GEMM_ROWS;
            s.variant = (n_gemm > 1 ? int(n_gemm) << 20 : 0) | (s.swiglu ? 1 << 29 : 0) | (s.norm_fused ? 1 << 30 : 0);
            if (s.norm_fused) {
              const Node& nn = p->nodes[s.nodes.back()];
              s.t_ptr[5] = nn.a; s.t_ptr[6] = nn.gamma; s.t_ptr[7] = nn.beta;
              s.norm_eps = (float)nn.eps;
              s.norm_x_f32 = p->wide[nn.a];
            }
            break;
          }
        }
        if (s.norm_fused) {
          set_error("step for op %d: the fused normalisation needs the few-row GEMM kernel", n.ops[0]);
          return FLUID_EUNSUPPORTED;
        }
        if (s.split_k > 1) {
          s.variant |= s.split_k << 24;
        } else if (s.kernel == FLUID_K_GEMM_TC && p->opts.split_k >= 0) {
          GemmParams gs[3] = {s.gemm, n_gemm > 1 ? s.gemm_x[0] : s.gemm, n_gemm > 2 ? s.gemm_x[1] : s.gemm};
          s.cluster_k = s.swiglu ? 0 : gemm_cluster_split(gs, s.tc, int(n_gemm));
          if (s.cluster_k > 1) s.variant |= (s.cluster_k << 24) | (1 << 28);
          else if (gemm_pair_eligible(gs, s.tc, int(n_gemm))) s.variant |= 1 << 29;
          if (s.swiglu && !((s.variant >> 29) & 1)) {
            set_error("step for op %d: the fused SwiGLU needs the CTA-pair form of the GEMM", n.ops[0]);
            return FLUID_EUNSUPPORTED;
          }
        }
        break;
      }
      case N_NORM: {
        s.kernel = FLUID_K_NORM;
        NormParams q{};
        q.dtype = ty.dtype;
        q.width = (int)ty.dims[ty.rank - 1];
        q.rows = int(ty.numel() / q.width);
        q.eps = (float)n.eps;
        q.rms = n.rms;
        q.x_f32 = p->wide[n.a];
        q.res_f32 = n.res >= 0 ? p->wide[n.res] : 0;
        s.norm = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.res; s.t_ptr[2] = n.gamma; s.t_ptr[3] = n.beta; s.t_ptr[4] = n.out;
        s.t_ptr[5] = n.out; s.t_narrow[5] = 1;  // bf16 copy of an fp32-held output, if one is planned
        {
          const double ne = (double)ty.numel();
          const bool twin = p->twin_record_of[p->alias_root[n.out]] >= 0;
          s.bytes = ne * (q.x_f32 ? 4.0 : es) + (n.res >= 0 ? ne * (q.res_f32 ? 4.0 : es) : 0.0) +
                    ne * (p->wide[n.out] ? 4.0 + (twin ? es : 0.0) : es);
        }
        break;
      }
      case N_SOFTMAX: {
        s.kernel = FLUID_K_SOFTMAX;
        SoftmaxParams q{};
        q.dtype = ty.dtype;
        q.n = (int)ty.dims[ty.rank - 1];
        q.rows = ty.numel() / q.n;
        q.rows_per_mat = ty.rank >= 2 ? (int)ty.dims[ty.rank - 2] : 1;
        q.scale = (float)n.scale;
        q.causal = n.sm_causal;
        q.zero_block = 0;
        if (q.causal) {  // zeros past the diagonal block are never read by k-clipped PV products
          bool all_clipped = true, any = false;
          for (const Step& s2 : p->steps)
            for (int nj : s2.nodes) {
              const Node& m = p->nodes[nj];
              for (int t : m.ins)
                if (p->alias_root[t] == p->alias_root[n.out]) {
                  any = true;
                  if (!(m.kind == N_GEMM && m.gemm_kind == G_PV && m.causal == CAUSAL_CLIP_K && m.a == t)) all_clipped = false;
                }
            }
          if (any && all_clipped && T[n.out].kind == FLUID_ACT) q.zero_block = 128;
        }
        s.softmax = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.out; s.t_narrow[0] = 1;
        double frac = 1.0;
        if (q.causal) frac = 0.5 * (1.0 + 1.0 / q.n);
        s.bytes = es * ty.numel() * 2.0 * frac;
        break;
      }
      case N_ROPE: {
        s.kernel = FLUID_K_ROPE;
        RopeParams q{};
        q.dtype = ty.dtype;
        int64_t st[FLUID_MAX_RANK];
        perm_strides(p, n.out, st);
        for (int i = 0; i < 4; ++i) {
          q.dims[i] = (int)ty.dims[i];
          q.st[i] = st[i];
          q.order[i] = p->cands[n.out][lo[n.out]][i];
        }
        rope_freq_fill(q.freq, n.rope_base, (int)ty.dims[3]);
        q.interleaved = n.rope_interleaved;
        q.pos_stride = (n.pos >= 0 && T[n.pos].dims[0] > 1) ? 1 : 0;
        s.rope = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.out; s.t_ptr[2] = n.pos; s.t_narrow[0] = 1;
        s.bytes = es * ty.numel() * 2.0;
        break;
      }
      case N_ELTWISE: {
        s.kernel = FLUID_K_ELTWISE;
        EltParams q{};
        q.dtype = ty.dtype;
        q.n = ty.numel();
        q.op = n.elt;
        if (n.elt == ELT_ADD) {  // a residual addition reads and writes the fp32 copies
          q.a_f32 = p->wide[n.a];
          q.b_f32 = n.b >= 0 ? p->wide[n.b] : 0;
        } else {
          s.t_narrow[0] = s.t_narrow[1] = 1;
        }
        q.y_f32 = p->wide[n.out];
        s.elt = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.b; s.t_ptr[2] = n.out;
        s.bytes = es * ty.numel() * (n.b >= 0 ? 3.0 : 2.0);
        break;
      }
      case N_TRANSPOSE: {
        s.kernel = FLUID_K_PERMUTE;
        PermuteParams q{};
        q.esize = (int)ty.esize();
        q.rank = ty.rank;
        int64_t sx[FLUID_MAX_RANK], sy[FLUID_MAX_RANK];
        perm_strides(p, n.a, sx);
        perm_strides(p, n.out, sy);
        q.x_inner = q.y_inner = -1;
        for (int j = 0; j < 5; ++j) {
          q.dims[j] = j < ty.rank ? (int)ty.dims[j] : 1;
          q.xs[j] = j < ty.rank ? sx[n.perm[j]] : 0;
          q.ys[j] = j < ty.rank ? sy[j] : 0;
          if (j < ty.rank && q.dims[j] > 1 && q.xs[j] == 1) q.x_inner = j;
          if (j < ty.rank && q.dims[j] > 1 && q.ys[j] == 1) q.y_inner = j;
        }
        s.permute = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.out; s.t_narrow[0] = 1;
        s.bytes = es * ty.numel() * 2.0;
        break;
      }
      case N_ATTN: {
        s.kernel = FLUID_K_ATTN;
        if (!lower_attn(p, n, lo, &s.attn, &s.attn_host)) {
          set_error("step for op %d: attention cannot be lowered under the chosen layouts", n.ops[0]);
          return FLUID_EUNSUPPORTED;
        }
        s.variant = s.attn.D | (s.attn.k_mn_major << 8) | (s.attn.v_k_major << 9) | (s.attn.causal << 10);
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.b; s.t_ptr[2] = n.v; s.t_ptr[3] = n.out;
        s.flops = 4.0 * s.attn.B * s.attn.NH * double(s.attn.S) * s.attn.S * s.attn.D * (s.attn.causal ? 0.5 * (1.0 + 1.0 / s.attn.S) : 1.0);
        s.bytes = es * (double(T[n.a].numel()) + T[n.b].numel() + T[n.v].numel() + ty.numel());
        break;
      }
      case N_ATTN_DECODE: {
        s.kernel = FLUID_K_ATTN_DECODE;
        AttnDecodeParams q{};
        const TensorDesc &tq = T[n.a], &tk = T[n.b], &tc = T[n.kc];
        q.dtype = ty.dtype;
        q.B = (int)tq.dims[0]; q.NH = (int)tq.dims[2]; q.NKV = (int)tk.dims[2]; q.D = (int)tq.dims[3]; q.Tmax = (int)tc.dims[1];
        q.scale_log2 = (float)(n.scale * 1.4426950408889634);
        q.rope = n.rope_fused;
        q.pos_stride = T[n.pos].dims[0] > 1 ? 1 : 0;
        rope_freq_fill(q.rope_freq, n.rope_base, q.D);
        int64_t st[FLUID_MAX_RANK];
        perm_strides(p, n.a, st);   q.q_sb = st[0]; q.q_sh = st[2];
        perm_strides(p, n.b, st);   q.k_sb = st[0]; q.k_sh = st[2];
        perm_strides(p, n.v, st);   q.v_sb = st[0]; q.v_sh = st[2];
        perm_strides(p, n.out, st); q.o_sb = st[0]; q.o_sh = st[2];
        s.attn_dec = q;
        s.variant = q.D | (q.NH / q.NKV) << 8 | q.rope << 16;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.b; s.t_ptr[2] = n.v; s.t_ptr[3] = n.kc; s.t_ptr[4] = n.vc; s.t_ptr[5] = n.pos;
        s.t_ptr[6] = n.out;
        // figures for a full cache; a run reads pos + 1 of its Tmax rows
        s.flops = 4.0 * q.B * q.NH * double(q.Tmax) * q.D;
        s.bytes = es * (double(T[n.kc].numel()) + T[n.vc].numel() + 2.0 * tq.numel() + 2.0 * tk.numel());
        break;
      }
      case N_SELECT: {
        s.kernel = FLUID_K_SELECT_LAST;
        const TensorDesc& tx = T[n.a];
        PermuteParams q{};
        q.esize = (int)ty.esize();
        q.rank = 2;
        for (int j = 0; j < 5; ++j) { q.dims[j] = 1; q.xs[j] = 0; q.ys[j] = 0; }
        q.dims[0] = (int)ty.dims[0]; q.dims[1] = (int)ty.dims[1];
        q.xs[0] = tx.dims[1] * tx.dims[2]; q.xs[1] = 1;
        q.ys[0] = ty.dims[1]; q.ys[1] = 1;
        q.x_offset = (tx.dims[1] - 1) * tx.dims[2];
        q.x_inner = q.y_inner = 1;
        s.permute = q;
        s.t_ptr[0] = n.a; s.t_ptr[1] = n.out;
        s.bytes = es * ty.numel() * 2.0;
        break;
      }
    }
  }
  return FLUID_OK;
}

struct Resolver {
  const fluid_plan_s* p;
  char* arena;
  const void* const* inputs;
  void* const* outputs;
  bool ok = true;
  const void* operator()(int t, int narrow = 0) {
    if (t < 0) return nullptr;
    const int r = p->alias_root[t];
    if (narrow && p->wide[r]) {
      const int rec = p->twin_record_of[r];
      if (rec < 0) {
        set_error("tensor %d has no bf16 copy", r);
        ok = false;
        return nullptr;
      }
      return arena + p->records[rec].offset;
    }
    const TensorDesc& td = p->graph.tensors[r];
    switch (td.kind) {
      case FLUID_INPUT:
      case FLUID_STATE: return inputs[p->input_slot[r]];
      case FLUID_OUTPUT: return outputs[p->output_slot[r]];
      case FLUID_CONST:
        if (!p->const_ptr[r]) {
          set_error("constant tensor %d is not bound", r);
          ok = false;
        }
        return p->const_ptr[r];
      default: {
        const int rec = p->record_of[r];
        if (rec < 0) {
          set_error("tensor %d has no storage", r);
          ok = false;
          return nullptr;
        }
        return arena + p->records[rec].offset;
      }
    }
  }
};

static int run_impl(fluid_plan_s* p, void* arena_ptr, const void* const* inputs, void* const* outputs,
                    cudaStream_t stream, float* step_ms) {
  if (!p || !arena_ptr) {
    set_error("null plan or arena");
    return FLUID_EINVAL;
  }
  if (reinterpret_cast<uintptr_t>(arena_ptr) % FLUID_ARENA_ALIGN) {
    set_error("arena_ptr must be %d-byte aligned", FLUID_ARENA_ALIGN);
    return FLUID_EALIGN;
  }
  if (p->not_runnable_op >= 0) {
    set_error("the plan's cost function chose layouts for op %d that no kernel runs: the plan can be inspected, not run",
              p->not_runnable_op);
    return FLUID_EUNSUPPORTED;
  }
  const auto& T = p->graph.tensors;
  std::vector<const void*> key;
  key.push_back(arena_ptr);
  for (int t = 0; t < (int)T.size(); ++t) {
    const void* q = nullptr;
    if (T[t].kind == FLUID_INPUT || T[t].kind == FLUID_STATE) {
      if (!inputs || !(q = inputs[p->input_slot[t]])) { set_error("input %d is null", p->input_slot[t]); return FLUID_EINVAL; }
    } else if (T[t].kind == FLUID_OUTPUT) {
      if (!outputs || !(q = outputs[p->output_slot[t]])) { set_error("output %d is null", p->output_slot[t]); return FLUID_EINVAL; }
    } else {
      continue;
    }
    if (reinterpret_cast<uintptr_t>(q) & 15) {
      set_error("input/output pointers must be 16-byte aligned");
      return FLUID_EALIGN;
    }
    key.push_back(q);
  }
  Resolver R{p, static_cast<char*>(arena_ptr), inputs, outputs};
  std::lock_guard<std::mutex> lk(p->mu);
  // tensor maps hold absolute addresses: (re-)encode when any base address changed
  if (!p->maps_valid || key != p->bound_key) {
    for (Step& s : p->steps) {
      if (s.kernel == FLUID_K_ATTN) {
        const void* q = R(s.t_ptr[0], 1);
        const void* k = R(s.t_ptr[1], 1);
        const void* v = R(s.t_ptr[2], 1);
        if (!R.ok) return FLUID_EINVAL;
        if (encode_tensor_map(&s.attn_host.map_q, q, s.attn_host.q) != 0 || encode_tensor_map(&s.attn_host.map_k, k, s.attn_host.k) != 0 ||
            encode_tensor_map(&s.attn_host.map_v, v, s.attn_host.v) != 0) {
          set_error("tensor map encoding failed for the attention step of op %d", p->nodes[s.node].ops[0]);
          return FLUID_ECUDA;
        }
        continue;
      }
      if (s.kernel != FLUID_K_GEMM_TC) continue;
      // (the second half of a split normalisation reads bf16(x * gain) from the scratch slice its producer filled)
      const void* a = s.nrm_pre ? static_cast<const void*>(static_cast<char*>(arena_ptr) + p->records[s.nrm_record].offset) : R(s.t_ptr[0], 1);
      const void* b = R(s.t_ptr[1], 1);
      if (!R.ok) return FLUID_EINVAL;
      bool enc_ok = encode_tensor_map(&s.tc.map_a, a, s.tc.a) == 0 && encode_tensor_map(&s.tc.map_b, b, s.tc.b) == 0;
      for (size_t gi = 1; enc_ok && gi < (s.swiglu ? size_t(2) : s.nodes.size() - s.rope_fused - s.nrm_pre); ++gi) {
        const void* bx = R(s.x_ptr[gi - 1][0], 1);
        if (!R.ok) return FLUID_EINVAL;
        enc_ok = encode_tensor_map(&s.tc_x[gi - 1].map_b, bx, s.tc_x[gi - 1].b) == 0;
      }
      if (!enc_ok) {
        set_error("tensor map encoding failed for the step of op %d", p->nodes[s.node].ops[0]);
        return FLUID_ECUDA;
      }
    }
    p->bound_key = key;
    p->maps_valid = true;
  }
  std::vector<cudaEvent_t> ev;
  if (step_ms) {
    ev.resize(p->steps.size() + 1);
    for (auto& e : ev) cudaEventCreate(&e);
    cudaEventRecord(ev[0], stream);
  }
  uint32_t* status = reinterpret_cast<uint32_t*>(arena_ptr);
  {  // the header's status words start every run at zero
    cudaError_t err = cudaMemsetAsync(arena_ptr, 0, FLUID_ARENA_HEADER, stream);
    if (err != cudaSuccess) {
      set_error("clearing the arena header: %s", cudaGetErrorString(err));
      return FLUID_ECUDA;
    }
  }
  int si = 0;
  for (Step& s : p->steps) {
    cudaError_t err = cudaSuccess;
    switch (s.kernel) {
      case FLUID_K_EMBED: {
        EmbedParams q = s.embed;
        q.ids = static_cast<const int*>(R(s.t_ptr[0])); q.tok = R(s.t_ptr[1]); q.pos = R(s.t_ptr[2]);
        q.y = const_cast<void*>(R(s.t_ptr[3]));
        q.pos_off = static_cast<const int*>(R(s.t_ptr[4]));
        if (R.ok) err = launch_embed(q, stream);
        break;
      }
      case FLUID_K_GEMM_SIMT:
      case FLUID_K_GEMM_TC: {
        GemmParams q = s.gemm;
        // split RMS normalisation: the scratch slice holds bf16(x * gain), then the slabs' sums of squares
        char* nrm_base = (s.nrm_emit || s.nrm_pre) ? static_cast<char*>(arena_ptr) + p->records[s.nrm_record].offset : nullptr;
        float* nrm_ss = nullptr;
        int nrm_slabs = 0;
        if (nrm_base) {
          const TensorDesc& tn = p->graph.tensors[p->nodes[s.nrm_node].out];
          nrm_ss = reinterpret_cast<float*>(static_cast<char*>(arena_ptr) + p->records[s.nrm_ss_record].offset);
          nrm_slabs = int(tn.dims[tn.rank - 1] / 128);
        }
        q.A = s.nrm_pre ? nrm_base : R(s.t_ptr[0], 1); q.B = R(s.t_ptr[1], 1); q.C = const_cast<void*>(R(s.t_ptr[2]));
        q.bias = R(s.t_ptr[3]); q.R = R(s.t_ptr[4]);
        if (s.nrm_emit) {
          q.nrm_out = nrm_base;
          q.nrm_gamma = R(p->nodes[s.nrm_node].gamma);
          q.nrm_ss = nrm_ss;
        }
        if (s.nrm_pre) {
          q.row_ss = nrm_ss;
          q.row_slabs = nrm_slabs;
          q.row_inv_n = 1.f / float(nrm_slabs * 128);
          q.row_eps = float(p->nodes[s.nrm_node].eps);
        }
        if (s.kernel == FLUID_K_GEMM_TC) {
          GemmParams gs[3] = {q, s.gemm_x[0], s.gemm_x[1]};
          GemmTcHost ts[3] = {s.tc, s.tc_x[0], s.tc_x[1]};
          const int ng = s.swiglu ? 2 : (int)s.nodes.size() - s.rope_fused - s.nrm_pre;
          for (int gi = 1; gi < ng; ++gi) {
            gs[gi].A = q.A;
            gs[gi].B = R(s.x_ptr[gi - 1][0], 1);
            gs[gi].C = s.swiglu ? q.C : const_cast<void*>(R(s.x_ptr[gi - 1][1]));
            gs[gi].bias = R(s.x_ptr[gi - 1][2]);
            gs[gi].R = nullptr;
            gs[gi].row_ss = q.row_ss; gs[gi].row_slabs = q.row_slabs; gs[gi].row_inv_n = q.row_inv_n; gs[gi].row_eps = q.row_eps;
          }
          float* partial = s.scratch_record >= 0
                               ? reinterpret_cast<float*>(static_cast<char*>(arena_ptr) + p->records[s.scratch_record].offset)
                               : nullptr;
          if (R.ok) err = launch_gemm_tc(gs, ts, ng, s.split_k, s.cluster_k, partial, status, stream, s.swiglu, s.rope_fused ? &s.rope_freq : nullptr);
        } else if (R.ok) {
          err = launch_gemm_simt(q, stream);
        }
        break;
      }
      case FLUID_K_GEMM_ROWS: {
        GemmParams gs[3] = {s.gemm, s.gemm_x[0], s.gemm_x[1]};
        const int ng = s.swiglu ? 2 : (int)s.nodes.size() - s.norm_fused;
        RowsNorm rn{};
        if (s.norm_fused) {
          rn.x = R(s.t_ptr[5]); rn.gamma = R(s.t_ptr[6]); rn.beta = R(s.t_ptr[7]); rn.eps = s.norm_eps; rn.x_f32 = s.norm_x_f32;
        }
        gs[0].A = s.norm_fused ? rn.x : R(s.t_ptr[0], 1); gs[0].B = R(s.t_ptr[1], 1); gs[0].C = const_cast<void*>(R(s.t_ptr[2]));
        gs[0].bias = R(s.t_ptr[3]); gs[0].R = R(s.t_ptr[4]);
        for (int gi = 1; gi < ng; ++gi) {
          gs[gi].A = gs[0].A;
          gs[gi].B = R(s.x_ptr[gi - 1][0], 1);
          gs[gi].C = s.swiglu ? gs[0].C : const_cast<void*>(R(s.x_ptr[gi - 1][1]));
          gs[gi].bias = R(s.x_ptr[gi - 1][2]);
          gs[gi].R = nullptr;
        }
        if (R.ok) err = launch_gemm_rows(gs, ng, stream, s.swiglu, s.norm_fused ? &rn : nullptr, status);
        break;
      }
      case FLUID_K_ATTN: {
        AttnParams q = s.attn;
        q.O = const_cast<void*>(R(s.t_ptr[3]));
        q.Q = R(s.t_ptr[0], 1); q.K = R(s.t_ptr[1], 1); q.V = R(s.t_ptr[2], 1);
        q.status = status;
        if (R.ok) err = launch_attn_tc(q, s.attn_host, stream);
        break;
      }
      case FLUID_K_NORM: {
        NormParams q = s.norm;
        q.x = R(s.t_ptr[0]); q.res = R(s.t_ptr[1]); q.gamma = R(s.t_ptr[2]); q.beta = R(s.t_ptr[3]);
        {
          const int out = s.t_ptr[4], root = p->alias_root[out];
          if (p->wide[root]) {
            q.y_hi = static_cast<float*>(const_cast<void*>(R(out)));
            q.y_lo = p->twin_record_of[root] >= 0 ? const_cast<void*>(R(out, 1)) : nullptr;
          } else if (p->graph.tensors[out].dtype == FLUID_F32) {
            q.y_hi = nullptr;
            q.y_lo = const_cast<void*>(R(out));
          } else {
            q.y_hi = nullptr;
            q.y_lo = const_cast<void*>(R(out));
          }
        }
        if (R.ok) err = launch_norm(q, stream);
        break;
      }
      case FLUID_K_SOFTMAX: {
        SoftmaxParams q = s.softmax;
        q.x = R(s.t_ptr[0], 1); q.y = const_cast<void*>(R(s.t_ptr[1]));
        if (R.ok) err = launch_softmax(q, stream);
        break;
      }
      case FLUID_K_ROPE: {
        RopeParams q = s.rope;
        q.x = R(s.t_ptr[0], 1); q.y = const_cast<void*>(R(s.t_ptr[1]));
        q.pos = static_cast<const int*>(R(s.t_ptr[2]));
        if (R.ok) err = launch_rope(q, stream);
        break;
      }
      case FLUID_K_ATTN_DECODE: {
        AttnDecodeParams q = s.attn_dec;
        q.q = R(s.t_ptr[0], 1); q.k = R(s.t_ptr[1], 1); q.v = R(s.t_ptr[2], 1);
        q.kc = const_cast<void*>(R(s.t_ptr[3])); q.vc = const_cast<void*>(R(s.t_ptr[4]));
        q.pos = static_cast<const int*>(R(s.t_ptr[5]));
        q.out = const_cast<void*>(R(s.t_ptr[6]));
        q.status = status;
        if (R.ok) err = launch_attn_decode(q, stream);
        break;
      }
      case FLUID_K_ELTWISE: {
        EltParams q = s.elt;
        q.a = R(s.t_ptr[0], s.t_narrow[0]); q.b = R(s.t_ptr[1], s.t_narrow[1]); q.y = const_cast<void*>(R(s.t_ptr[2]));
        if (R.ok) err = launch_eltwise(q, stream);
        break;
      }
      case FLUID_K_PERMUTE:
      case FLUID_K_SELECT_LAST: {
        PermuteParams q = s.permute;
        q.x = R(s.t_ptr[0], 1); q.y = const_cast<void*>(R(s.t_ptr[1]));
        q.status = status;
        if (R.ok) err = launch_permute(q, stream);
        break;
      }
    }
    if (!R.ok) return FLUID_EINVAL;
    if (err != cudaSuccess) {
      set_error("step %d (kernel %d): %s", si, s.kernel, cudaGetErrorString(err));
      return FLUID_ECUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    ++si;
    if (step_ms) cudaEventRecord(ev[si], stream);
  }
  if (step_ms) {
    cudaError_t err = cudaStreamSynchronize(stream);
    for (size_t i = 0; i + 1 < ev.size(); ++i) {
      float ms = 0;
      cudaEventElapsedTime(&ms, ev[i], ev[i + 1]);
      step_ms[i] = ms;
    }
    for (auto& e : ev) cudaEventDestroy(e);
    if (err != cudaSuccess) {
      set_error("stream synchronise: %s", cudaGetErrorString(err));
      return FLUID_ECUDA;
    }
  }
  return FLUID_OK;
}

int pack_constant_launch(const fluid_plan_s* p, int t, const void* src, void* dst, void* stream) {
  const TensorDesc& td = p->graph.tensors[t];
  PermuteParams q{};
  q.esize = (int)td.esize();
  q.rank = td.rank;
  int64_t sx[FLUID_MAX_RANK], sy[FLUID_MAX_RANK];
  strides_of(td, identity_perm(), sx);
  strides_of(td, p->cands[t][p->layout[t]], sy);
  q.x_inner = q.y_inner = -1;
  for (int j = 0; j < 5; ++j) {
    q.dims[j] = j < td.rank ? (int)td.dims[j] : 1;
    q.xs[j] = j < td.rank ? sx[j] : 0;
    q.ys[j] = j < td.rank ? sy[j] : 0;
    if (j < td.rank && q.dims[j] > 1 && q.xs[j] == 1) q.x_inner = j;
    if (j < td.rank && q.dims[j] > 1 && q.ys[j] == 1) q.y_inner = j;
  }
  q.x = src;
  q.y = dst;
  cudaError_t err = launch_permute(q, static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) {
    set_error("pack_constant: %s", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return FLUID_OK;
}

}  // namespace fluid

using namespace fluid;

extern "C" {

int fluid_run(fluid_plan_t* plan, void* arena_ptr, const void* const* inputs, void* const* outputs,
              fluid_stream stream) {
  return run_impl(plan, arena_ptr, inputs, outputs, static_cast<cudaStream_t>(stream), nullptr);
}

int fluid_run_profiled(fluid_plan_t* plan, void* arena_ptr, const void* const* inputs, void* const* outputs,
                       fluid_stream stream, float* step_ms) {
  if (!step_ms) {
    set_error("step_ms is null");
    return FLUID_EINVAL;
  }
  return run_impl(plan, arena_ptr, inputs, outputs, static_cast<cudaStream_t>(stream), step_ms);
}

int fluid_pack_constant(const fluid_plan_t* plan, int tensor_id, const void* dev_src_canonical, void* dev_dst,
                        fluid_stream stream) {
  if (!plan || tensor_id < 0 || tensor_id >= (int)plan->graph.tensors.size() || !dev_src_canonical || !dev_dst) {
    set_error("pack_constant: bad argument");
    return FLUID_EINVAL;
  }
  return pack_constant_launch(plan, tensor_id, dev_src_canonical, dev_dst, stream);
}

int fluid_status(const fluid_plan_t* plan, const void* arena_ptr, fluid_stream stream, int* device_status) {
  if (!plan || !arena_ptr || !device_status) {
    set_error("status: null argument");
    return FLUID_EINVAL;
  }
  uint32_t word = 0;
  cudaError_t err = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (err == cudaSuccess) err = cudaMemcpy(&word, arena_ptr, sizeof(word), cudaMemcpyDeviceToHost);
  if (err != cudaSuccess) {
    set_error("status: %s", cudaGetErrorString(err));
    return FLUID_ECUDA;
  }
  *device_status = (int)word;
  if (word & 0x10u) {
    set_error("CACHED_ATTENTION: the position read on the device lies outside the cache (status 0x%x)", word);
    return FLUID_EINVAL;
  }
  if (word != 0) {
    set_error("a device-side wait expired (code 0x%x)", word);
    return FLUID_ETIMEOUT;
  }
  return FLUID_OK;
}

int64_t fluid_launch_count(void) { return g_launches.load(); }

}  // extern "C"
