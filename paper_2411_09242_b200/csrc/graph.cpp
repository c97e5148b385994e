// Graph construction and shape checking (host only).
#include <cstdarg>
#include <cstdio>
#include <new>

#include "fluid_internal.h"

namespace fluid {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

static bool same_dims(const TensorDesc& a, const TensorDesc& b) {
  if (a.rank != b.rank) return false;
  for (int i = 0; i < a.rank; ++i)
    if (a.dims[i] != b.dims[i]) return false;
  return true;
}

static int check_op(const fluid_graph_s* g, const OpDesc& op) {
  auto T = [&](int id) -> const TensorDesc& { return g->tensors[id]; };
  auto need = [&](bool ok, const char* what) {
    if (!ok) set_error("op %d: %s", op.kind, what);
    return ok;
  };
  const int ni = (int)op.ins.size(), no = (int)op.outs.size();
  if (!need(no == 1, "exactly one output expected")) return FLUID_EINVAL;
  const TensorDesc& y = T(op.outs[0]);
  if (!need(y.kind == FLUID_ACT || y.kind == FLUID_OUTPUT, "an op may only write ACT or OUTPUT tensors"))
    return FLUID_EINVAL;
  for (int i = 0; i < ni; ++i)
    if (T(op.ins[i]).kind == FLUID_STATE && !(op.kind == FLUID_OP_CACHED_ATTENTION && (i == 3 || i == 4))) {
      need(false, "a STATE tensor is read only as the cache of a CACHED_ATTENTION op");
      return FLUID_EINVAL;
    }
  switch (op.kind) {
    case FLUID_OP_EMBED: {
      if (!need(ni >= 2 && ni <= 4, "EMBED takes ids, table [, positions [, offset]]")) return FLUID_EINVAL;
      const TensorDesc &ids = T(op.ins[0]), &tok = T(op.ins[1]);
      bool ok = ids.dtype == FLUID_I32 && ids.rank == 2 && tok.rank == 2 && y.rank == 3 &&
                y.dims[0] == ids.dims[0] && y.dims[1] == ids.dims[1] && y.dims[2] == tok.dims[1] &&
                tok.dtype == y.dtype;
      if (ok && ni >= 3) {
        const TensorDesc& pos = T(op.ins[2]);
        ok = pos.rank == 2 && pos.dims[0] >= ids.dims[1] && pos.dims[1] == tok.dims[1] && pos.dtype == y.dtype;
      }
      if (ok && ni == 4) {
        const TensorDesc& off = T(op.ins[3]);
        ok = off.dtype == FLUID_I32 && off.rank == 1 && (off.dims[0] == 1 || off.dims[0] == ids.dims[0]) && off.kind == FLUID_INPUT;
      }
      if (!need(ok, "EMBED shapes")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_LINEAR: {
      if (!need(ni == 2 || ni == 3, "LINEAR takes x, w [, bias]")) return FLUID_EINVAL;
      const TensorDesc &x = T(op.ins[0]), &w = T(op.ins[1]);
      const int c = op.attrs.contract;
      bool ok = c >= 1 && c < x.rank + 1 && c < w.rank && x.rank - c >= 1 && x.dtype == w.dtype && x.dtype == y.dtype &&
                x.dtype != FLUID_I32;
      if (ok)
        for (int i = 0; i < c; ++i) ok = ok && x.dims[x.rank - c + i] == w.dims[i];
      ok = ok && y.rank == (x.rank - c) + (w.rank - c);
      if (ok) {
        for (int i = 0; i < x.rank - c; ++i) ok = ok && y.dims[i] == x.dims[i];
        for (int i = 0; i < w.rank - c; ++i) ok = ok && y.dims[x.rank - c + i] == w.dims[c + i];
      }
      if (ok && ni == 3) {
        const TensorDesc& b = T(op.ins[2]);
        ok = b.rank == w.rank - c && b.dtype == y.dtype;
        if (ok)
          for (int i = 0; i < b.rank; ++i) ok = ok && b.dims[i] == w.dims[c + i];
      }
      if (!need(ok, "LINEAR shapes")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_ADD:
    case FLUID_OP_MUL:
      if (!need(ni == 2 && same_dims(T(op.ins[0]), y) && same_dims(T(op.ins[1]), y) &&
                    T(op.ins[0]).dtype == y.dtype && T(op.ins[1]).dtype == y.dtype && y.dtype != FLUID_I32,
                "binary elementwise shapes"))
        return FLUID_EINVAL;
      break;
    case FLUID_OP_GELU:
    case FLUID_OP_SILU:
    case FLUID_OP_SOFTMAX:
      if (!need(ni == 1 && same_dims(T(op.ins[0]), y) && T(op.ins[0]).dtype == y.dtype && y.dtype != FLUID_I32,
                "unary op shapes"))
        return FLUID_EINVAL;
      if (op.kind == FLUID_OP_SOFTMAX && op.attrs.causal && !need(y.rank >= 2, "causal SOFTMAX needs rank >= 2"))
        return FLUID_EINVAL;
      break;
    case FLUID_OP_LAYERNORM:
    case FLUID_OP_RMSNORM: {
      const int want = op.kind == FLUID_OP_LAYERNORM ? 3 : 2;
      bool ok = ni == want && same_dims(T(op.ins[0]), y) && T(op.ins[0]).dtype == y.dtype && y.dtype != FLUID_I32;
      for (int i = 1; ok && i < want; ++i)
        ok = T(op.ins[i]).rank == 1 && T(op.ins[i]).dims[0] == y.dims[y.rank - 1] && T(op.ins[i]).dtype == y.dtype;
      if (!need(ok, "norm shapes")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_ROPE:
      if (!need((ni == 1 || ni == 2) && y.rank == 4 && same_dims(T(op.ins[0]), y) && T(op.ins[0]).dtype == y.dtype &&
                    y.dims[3] % 2 == 0 && y.dtype != FLUID_I32,
                "ROPE wants x[B,S,nh,D] with even D"))
        return FLUID_EINVAL;
      if (ni == 2 && !need(T(op.ins[1]).dtype == FLUID_I32 && T(op.ins[1]).rank == 1 &&
                               (T(op.ins[1]).dims[0] == 1 || T(op.ins[1]).dims[0] == y.dims[0]) && T(op.ins[1]).kind == FLUID_INPUT,
                           "ROPE's position offset is an int32 [1] or [B] graph input"))
        return FLUID_EINVAL;
      break;
    case FLUID_OP_CACHED_ATTENTION: {
      bool ok = ni == 6;
      if (ok) {
        const TensorDesc &q = T(op.ins[0]), &k = T(op.ins[1]), &v = T(op.ins[2]), &kc = T(op.ins[3]), &vc = T(op.ins[4]),
                         &pos = T(op.ins[5]);
        ok = q.rank == 4 && same_dims(q, y) && q.dims[1] == 1 && k.rank == 4 && same_dims(k, v) && k.dims[0] == q.dims[0] &&
             k.dims[1] == 1 && k.dims[3] == q.dims[3] && q.dims[2] % k.dims[2] == 0 && kc.rank == 4 && same_dims(kc, vc) &&
             kc.dims[0] == q.dims[0] && kc.dims[2] == k.dims[2] && kc.dims[3] == q.dims[3] && kc.kind == FLUID_STATE &&
             vc.kind == FLUID_STATE && op.ins[3] != op.ins[4] && pos.dtype == FLUID_I32 && pos.rank == 1 &&
             (pos.dims[0] == 1 || pos.dims[0] == q.dims[0]) && pos.kind == FLUID_INPUT && y.dtype != FLUID_I32 && q.dtype == y.dtype && k.dtype == y.dtype &&
             v.dtype == y.dtype && kc.dtype == y.dtype && vc.dtype == y.dtype;
      }
      if (!need(ok, "CACHED_ATTENTION wants q[B,1,nh,D], k, v[B,1,nkv,D], two STATE caches [B,Tmax,nkv,D], pos i32[1] or [B]"))
        return FLUID_EINVAL;
      for (const OpDesc& o : g->ops)
        if (o.kind == FLUID_OP_CACHED_ATTENTION)
          for (int s = 3; s <= 4; ++s)
            if (!need(o.ins[3] != op.ins[s] && o.ins[4] != op.ins[s], "a cache belongs to one CACHED_ATTENTION op"))
              return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_TRANSPOSE: {
      const TensorDesc& x = T(op.ins.empty() ? op.outs[0] : op.ins[0]);
      bool ok = ni == 1 && x.rank == y.rank && x.dtype == y.dtype;
      int seen = 0;
      for (int i = 0; ok && i < y.rank; ++i) {
        const int p = op.attrs.perm[i];
        ok = p >= 0 && p < x.rank && !(seen & (1 << p)) && y.dims[i] == x.dims[p];
        seen |= 1 << p;
      }
      if (!need(ok, "TRANSPOSE perm / shapes")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_BMM_QK: {
      bool ok = ni == 2;
      if (ok) {
        const TensorDesc &q = T(op.ins[0]), &k = T(op.ins[1]);
        ok = q.rank == 4 && k.rank == 4 && y.rank == 4 && q.dims[0] == k.dims[0] && q.dims[1] == k.dims[1] &&
             q.dims[3] == k.dims[2] && y.dims[0] == q.dims[0] && y.dims[1] == q.dims[1] && y.dims[2] == q.dims[2] &&
             y.dims[3] == k.dims[3] && q.dtype == k.dtype && q.dtype == y.dtype && y.dtype != FLUID_I32;
      }
      if (!need(ok, "BMM_QK wants q[B,nh,S,D], kt[B,nh,D,S] -> [B,nh,S,S]")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_BMM_PV: {
      bool ok = ni == 2;
      if (ok) {
        const TensorDesc &p = T(op.ins[0]), &v = T(op.ins[1]);
        ok = p.rank == 4 && v.rank == 4 && y.rank == 4 && p.dims[0] == v.dims[0] && p.dims[1] == v.dims[1] &&
             p.dims[3] == v.dims[2] && y.dims[0] == p.dims[0] && y.dims[1] == p.dims[1] && y.dims[2] == p.dims[2] &&
             y.dims[3] == v.dims[3] && p.dtype == v.dtype && p.dtype == y.dtype && y.dtype != FLUID_I32;
      }
      if (!need(ok, "BMM_PV wants p[B,nh,S,S], v[B,nh,S,D] -> [B,nh,S,D]")) return FLUID_EINVAL;
      break;
    }
    case FLUID_OP_SELECT_LAST_TOKEN: {
      bool ok = ni == 1 && T(op.ins[0]).rank == 3 && y.rank == 2 && y.dims[0] == T(op.ins[0]).dims[0] &&
                y.dims[1] == T(op.ins[0]).dims[2] && y.dtype == T(op.ins[0]).dtype;
      if (!need(ok, "SELECT_LAST_TOKEN wants x[B,S,H] -> [B,H]")) return FLUID_EINVAL;
      break;
    }
    default:
      set_error("unknown op kind %d", op.kind);
      return FLUID_EINVAL;
  }
  return FLUID_OK;
}

}  // namespace fluid

using namespace fluid;

extern "C" {

const char* fluid_last_error(void) { return g_err; }

int fluid_graph_create(fluid_graph_t** g) {
  if (!g) {
    set_error("null out pointer");
    return FLUID_EINVAL;
  }
  *g = new (std::nothrow) fluid_graph_s();
  if (!*g) {
    set_error("out of host memory");
    return FLUID_ENOMEM;
  }
  return FLUID_OK;
}

void fluid_graph_destroy(fluid_graph_t* g) { delete g; }

int fluid_graph_add_tensor(fluid_graph_t* g, int dtype, int rank, const int64_t* dims, int kind, int* tensor_id) {
  if (!g || !dims || !tensor_id) {
    set_error("null argument");
    return FLUID_EINVAL;
  }
  if (dtype < FLUID_F32 || dtype > FLUID_I32 || kind < FLUID_INPUT || kind > FLUID_STATE || rank < 1 ||
      rank > FLUID_MAX_RANK) {
    set_error("bad dtype/kind/rank (%d/%d/%d)", dtype, kind, rank);
    return FLUID_EINVAL;
  }
  TensorDesc t;
  t.dtype = dtype;
  t.rank = rank;
  t.kind = kind;
  int64_t n = 1;
  for (int i = 0; i < rank; ++i) {
    if (dims[i] < 1 || dims[i] > (int64_t(1) << 31) - 1) {
      set_error("dim %d = %lld out of range", i, (long long)dims[i]);
      return FLUID_EINVAL;
    }
    t.dims[i] = dims[i];
    n *= dims[i];
    if (n > (int64_t(1) << 40)) {
      set_error("tensor too large");
      return FLUID_EINVAL;
    }
  }
  g->tensors.push_back(t);
  *tensor_id = (int)g->tensors.size() - 1;
  return FLUID_OK;
}

int fluid_graph_add_op(fluid_graph_t* g, int op_kind, int n_in, const int* in_ids, int n_out, const int* out_ids,
                       const fluid_op_attrs* attrs, int* op_id) {
  if (!g || (n_in > 0 && !in_ids) || !out_ids) {
    set_error("null argument");
    return FLUID_EINVAL;
  }
  if (op_kind < 0 || op_kind >= FLUID_OP_COUNT || n_in < 1 || n_in > 6 || n_out != 1) {
    set_error("bad op kind or arity (%d, %d in, %d out)", op_kind, n_in, n_out);
    return FLUID_EINVAL;
  }
  OpDesc op;
  op.kind = op_kind;
  const int nt = (int)g->tensors.size();
  for (int i = 0; i < n_in; ++i) {
    if (in_ids[i] < 0 || in_ids[i] >= nt) {
      set_error("input tensor id %d out of range", in_ids[i]);
      return FLUID_EINVAL;
    }
    op.ins.push_back(in_ids[i]);
  }
  for (int i = 0; i < n_out; ++i) {
    if (out_ids[i] < 0 || out_ids[i] >= nt) {
      set_error("output tensor id %d out of range", out_ids[i]);
      return FLUID_EINVAL;
    }
    for (const OpDesc& o : g->ops)
      for (int t : o.outs)
        if (t == out_ids[i]) {
          set_error("tensor %d already has a producer", t);
          return FLUID_EINVAL;
        }
    op.outs.push_back(out_ids[i]);
  }
  if (attrs) op.attrs = *attrs;
  if (op.attrs.contract == 0) op.attrs.contract = 1;
  if (op.attrs.scale == 0.0) op.attrs.scale = 1.0;
  if (op.attrs.eps == 0.0) op.attrs.eps = 1e-5;
  if (op.attrs.rope_base == 0.0) op.attrs.rope_base = 10000.0;
  int rc = check_op(g, op);
  if (rc != FLUID_OK) return rc;
  g->ops.push_back(op);
  if (op_id) *op_id = (int)g->ops.size() - 1;
  return FLUID_OK;
}

}  // extern "C"
