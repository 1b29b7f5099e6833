// Epilogue programs given as data: host-side analysis and lowering (Sec. 5.2 frontend mapping, Sec. 5.3 reduction
// subgraph splitting, Sec. 5.4 backend mapping) and the entry points that run them.
//
//   analyse():  checks the node list (closed vocabulary, edges to earlier nodes only, consistent parameter use), types
//               every node (tensor / per-row / constant), folds constants, marks what the terminal and the row outputs
//               depend on, and numbers the stages: a reduction's result belongs to the stage after its input's.
//   match_*():  canonicalisation onto the compiled fused instantiations.  The matchers walk the DAG from the terminal
//               node and accept any operand order of commutative nodes and any subset of the optional nodes.
//   lower_row_program(): the standard pathway -- one instruction per live computed node, shared-memory slots assigned
//               by liveness (a node's buffer is released at its last use and may be overwritten in place).
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "comfuse.h"
#include "fusion_spec.h"
#include "host_common.h"

namespace comfuse {

namespace {

enum NodeType : uint8_t { T_TENSOR = 0, T_ROW = 1, T_CONST = 2 };

bool is_unary(int op) { return op >= COMFUSE_OP_NEG && op <= COMFUSE_OP_SIGMOID; }
bool is_binary(int op) { return op >= COMFUSE_OP_ADD && op <= COMFUSE_OP_MIN; }
bool is_reduce(int op) { return op >= COMFUSE_OP_RED_SUM && op <= COMFUSE_OP_RED_TOPK_INDICES; }
bool is_topk(int op) { return op == COMFUSE_OP_RED_TOPK_VALUES || op == COMFUSE_OP_RED_TOPK_INDICES; }
bool is_leaf(int op) { return op >= COMFUSE_OP_ACC && op <= COMFUSE_OP_CAUSAL_MASK; }

float fold_unary(int op, float a) {
  switch (op) {
    case COMFUSE_OP_NEG: return -a;
    case COMFUSE_OP_ABS: return std::fabs(a);
    case COMFUSE_OP_SQUARE: return a * a;
    case COMFUSE_OP_SQRT: return std::sqrt(a);
    case COMFUSE_OP_RSQRT: return 1.f / std::sqrt(a);
    case COMFUSE_OP_RECIP: return 1.f / a;
    case COMFUSE_OP_EXP: return std::exp(a);
    case COMFUSE_OP_LOG: return std::log(a);
    case COMFUSE_OP_TANH: return std::tanh(a);
    case COMFUSE_OP_RELU: return a > 0.f ? a : 0.f;
    case COMFUSE_OP_GELU_TANH: return 0.5f * a * (1.f + std::tanh(0.7978845608028654f * (a + 0.044715f * a * a * a)));
    case COMFUSE_OP_SIGMOID: return 1.f / (1.f + std::exp(-a));
    default: return a;
  }
}

float fold_binary(int op, float a, float b) {
  switch (op) {
    case COMFUSE_OP_ADD: return a + b;
    case COMFUSE_OP_SUB: return a - b;
    case COMFUSE_OP_MUL: return a * b;
    case COMFUSE_OP_DIV: return a / b;
    case COMFUSE_OP_MAX: return a > b ? a : b;
    case COMFUSE_OP_MIN: return a < b ? a : b;
    default: return a;
  }
}

struct Analysis {
  int n = 0;
  std::vector<comfuse_spec_node_t> nodes;
  std::vector<uint8_t> type;     // NodeType
  std::vector<float> cval;       // value of T_CONST nodes (given or folded)
  std::vector<uint8_t> live;
  std::vector<int> stage;
  int param_kind[COMFUSE_SPEC_MAX_PARAMS];  // 0 unused, COMFUSE_OP_ROWVEC or COMFUSE_OP_TENSOR
  int terminal = 0;
  std::vector<int> row_outputs;
  int n_stages = 1, n_reductions = 0, n_live = 0;
};

comfuse_status_t analyse(const comfuse_fusion_spec_t* spec, Analysis& an) {
  if (!spec || !spec->nodes) return COMFUSE_ERR_INVALID_ARG;
  if (spec->n_nodes < 1 || spec->n_nodes > COMFUSE_SPEC_MAX_NODES) return COMFUSE_ERR_INVALID_ARG;
  if (spec->n_params < 0 || spec->n_params > COMFUSE_SPEC_MAX_PARAMS) return COMFUSE_ERR_INVALID_ARG;
  if (spec->n_row_outputs < 0 || spec->n_row_outputs > COMFUSE_SPEC_MAX_ROW_OUTPUTS) return COMFUSE_ERR_INVALID_ARG;
  if (spec->n_row_outputs > 0 && !spec->row_outputs) return COMFUSE_ERR_INVALID_ARG;
  if (spec->terminal < 0 || spec->terminal >= spec->n_nodes) return COMFUSE_ERR_INVALID_ARG;
  if (is_topk(spec->nodes[spec->terminal].op)) return COMFUSE_ERR_INVALID_ARG;
  const int n = spec->n_nodes;
  an.n = n;
  an.nodes.assign(spec->nodes, spec->nodes + n);
  an.type.assign(n, T_TENSOR);
  an.cval.assign(n, 0.f);
  an.live.assign(n, 0);
  an.stage.assign(n, 0);
  an.terminal = spec->terminal;
  std::memset(an.param_kind, 0, sizeof(an.param_kind));
  for (int k = 0; k < n; ++k) {
    const comfuse_spec_node_t& nd = an.nodes[k];
    const int op = nd.op;
    auto edge_ok = [&](int e) { return e >= 0 && e < k; };
    if (is_leaf(op)) {
      if (nd.in0 != -1 || nd.in1 != -1) return COMFUSE_ERR_INVALID_ARG;
      if (op == COMFUSE_OP_ROWVEC || op == COMFUSE_OP_TENSOR) {
        if (nd.param < 0 || nd.param >= spec->n_params) return COMFUSE_ERR_INVALID_ARG;
        if (an.param_kind[nd.param] != 0 && an.param_kind[nd.param] != op) return COMFUSE_ERR_INVALID_ARG;  // one slot, two shapes
        an.param_kind[nd.param] = op;
      } else if (nd.param != -1) {
        return COMFUSE_ERR_INVALID_ARG;
      }
      if (op == COMFUSE_OP_CONST) {
        an.type[k] = T_CONST;
        an.cval[k] = nd.imm;
      }
    } else if (is_unary(op) || is_reduce(op)) {
      if (!edge_ok(nd.in0) || nd.in1 != -1) return COMFUSE_ERR_INVALID_ARG;
      if (is_topk(op) ? (nd.param < 1 || nd.param > 64) : nd.param != -1) return COMFUSE_ERR_INVALID_ARG;
      if (is_topk(an.nodes[nd.in0].op)) return COMFUSE_ERR_INVALID_ARG;  // K values per row: a row output only
      if (is_reduce(op)) {
        an.type[k] = T_ROW;
        an.stage[k] = an.stage[nd.in0] + 1;
      } else {
        an.type[k] = an.type[nd.in0];
        an.stage[k] = an.stage[nd.in0];
        if (an.type[k] == T_CONST) an.cval[k] = fold_unary(op, an.cval[nd.in0]);
      }
    } else if (is_binary(op)) {
      if (!edge_ok(nd.in0) || !edge_ok(nd.in1) || nd.param != -1) return COMFUSE_ERR_INVALID_ARG;
      if (is_topk(an.nodes[nd.in0].op) || is_topk(an.nodes[nd.in1].op)) return COMFUSE_ERR_INVALID_ARG;
      const uint8_t ta = an.type[nd.in0], tb = an.type[nd.in1];
      an.type[k] = (ta == T_TENSOR || tb == T_TENSOR) ? T_TENSOR : (ta == T_ROW || tb == T_ROW) ? T_ROW : T_CONST;
      an.stage[k] = an.stage[nd.in0] > an.stage[nd.in1] ? an.stage[nd.in0] : an.stage[nd.in1];
      if (an.type[k] == T_CONST) an.cval[k] = fold_binary(op, an.cval[nd.in0], an.cval[nd.in1]);
    } else {
      return COMFUSE_ERR_INVALID_ARG;  // outside the vocabulary: rejected, never dropped
    }
  }
  an.row_outputs.assign(spec->row_outputs, spec->row_outputs + spec->n_row_outputs);
  for (int r : an.row_outputs) {
    if (r < 0 || r >= n) return COMFUSE_ERR_INVALID_ARG;
    if (an.type[r] == T_TENSOR) return COMFUSE_ERR_INVALID_ARG;  // a row output is one value per row
  }
  // liveness: what the terminal and the row outputs depend on (constants that were folded need no inputs)
  an.live[an.terminal] = 1;
  for (int r : an.row_outputs) an.live[r] = 1;
  for (int k = n - 1; k >= 0; --k) {
    if (!an.live[k] || an.type[k] == T_CONST) continue;
    if (an.nodes[k].in0 >= 0) an.live[an.nodes[k].in0] = 1;
    if (an.nodes[k].in1 >= 0) an.live[an.nodes[k].in1] = 1;
  }
  int max_stage = 0;
  for (int k = 0; k < n; ++k) {
    if (!an.live[k]) continue;
    ++an.n_live;
    if (is_reduce(an.nodes[k].op)) ++an.n_reductions;
    if (an.stage[k] > max_stage) max_stage = an.stage[k];
  }
  an.n_stages = max_stage + 1;
  return COMFUSE_OK;
}

// ------------------------------------------------------------------------------------------------ canonicalisation
struct FusedMatch {
  int kind = -1;
  uint32_t flags = 0;
  float alpha = 1.f, eps = 0.f, softcap = 0.f;
  int causal = 0;
  int bias = -1, residual = -1, gamma = -1, beta = -1;  // parameter slots, -1 = absent
  int row_max_out = -1, row_argmax_out = -1;            // positions in row_outputs, -1 = not asked for
  int activation = 0;                                   // BIAS_ACTIVATION kind: comfuse_op_t of the unary node, 0 = none
};

struct Matcher {
  const Analysis& an;
  std::vector<uint8_t> used;
  explicit Matcher(const Analysis& a) : an(a), used(a.n, 0) {}
  const comfuse_spec_node_t& nd(int k) const { return an.nodes[k]; }
  bool is(int k, int op) const { return k >= 0 && an.type[k] != T_CONST && nd(k).op == op; }
  bool is_const(int k) const { return k >= 0 && an.type[k] == T_CONST; }
  void use(int k) { used[k] = 1; }
  // binary node `k` of kind `op` with one operand satisfying `pred`: returns the OTHER operand and the matching one
  template <class Pred>
  bool split(int k, int op, Pred pred, int& other, int& hit) const {
    if (!is(k, op)) return false;
    const int a = nd(k).in0, b = nd(k).in1;
    if (pred(b)) { other = a; hit = b; return true; }
    if (op != COMFUSE_OP_SUB && op != COMFUSE_OP_DIV && pred(a)) { other = b; hit = a; return true; }
    return false;
  }
  bool all_live_used() const {
    for (int k = 0; k < an.n; ++k)
      if (an.live[k] && !used[k] && an.type[k] != T_CONST) return false;
    return true;
  }

  // x = [act](alpha * acc [+ bias]) [+ residual], peeled from the outside; without an activation the bias and the
  // residual may come in either order (with one, gelu_entry_order_ok() checks the order afterwards)
  bool entry(int k, bool allow_act, FusedMatch& m, bool& had_act) {
    had_act = false;
    int other, hit;
    for (int guard = 0; guard < 4; ++guard) {
      if (m.residual < 0 && split(k, COMFUSE_OP_ADD, [&](int t) { return is(t, COMFUSE_OP_TENSOR); }, other, hit)) {
        m.residual = nd(hit).param; use(k); use(hit); k = other;
      } else if (!had_act && allow_act && is(k, COMFUSE_OP_GELU_TANH)) {
        had_act = true; use(k); k = nd(k).in0;
      } else if (m.bias < 0 && split(k, COMFUSE_OP_ADD, [&](int t) { return is(t, COMFUSE_OP_ROWVEC); }, other, hit)) {
        m.bias = nd(hit).param; use(k); use(hit); k = other;
      } else {
        break;
      }
    }
    if (split(k, COMFUSE_OP_MUL, [&](int t) { return is_const(t); }, other, hit)) {
      m.alpha = an.cval[hit]; use(k); k = other;
    }
    if (!is(k, COMFUSE_OP_ACC)) return false;
    use(k);
    return true;
  }
};

// Order check for the GELU entry: residual outside the activation, bias inside (entry() peels greedily).
bool gelu_entry_order_ok(const Analysis& an, int x) {
  // chain from x down to acc: ops seen in order
  int k = x;
  bool seen_act = false;
  for (int guard = 0; guard < 8; ++guard) {
    const comfuse_spec_node_t& nd = an.nodes[k];
    if (nd.op == COMFUSE_OP_ACC) return true;
    if (nd.op == COMFUSE_OP_GELU_TANH) { seen_act = true; k = nd.in0; continue; }
    if (nd.op == COMFUSE_OP_ADD || nd.op == COMFUSE_OP_MUL) {
      const int a = nd.in0, b = nd.in1;
      const bool a_leaf = is_leaf(an.nodes[a].op) && an.nodes[a].op != COMFUSE_OP_ACC, b_leaf = is_leaf(an.nodes[b].op) && an.nodes[b].op != COMFUSE_OP_ACC;
      const int leaf = b_leaf ? b : a_leaf ? a : -1;
      if (leaf < 0) return false;
      const int lop = an.nodes[leaf].op;
      if (lop == COMFUSE_OP_TENSOR && seen_act) return false;   // residual inside the activation
      if (lop == COMFUSE_OP_ROWVEC && !seen_act) return false;  // bias outside the activation
      k = leaf == b ? a : b;
      continue;
    }
    return false;
  }
  return false;
}

bool match_layernorm(const Analysis& an, FusedMatch& m) {
  if (!an.row_outputs.empty()) return false;
  Matcher t(an);
  int k = an.terminal, other, hit;
  if (t.is(k, COMFUSE_OP_RELU)) { m.flags |= COMFUSE_FLAG_POST_RELU; t.use(k); k = t.nd(k).in0; }
  if (t.split(k, COMFUSE_OP_ADD, [&](int q) { return t.is(q, COMFUSE_OP_ROWVEC); }, other, hit)) {
    m.beta = t.nd(hit).param; t.use(k); t.use(hit); k = other;
  }
  if (t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is(q, COMFUSE_OP_ROWVEC); }, other, hit)) {
    m.gamma = t.nd(hit).param; t.use(k); t.use(hit); k = other;
  }
  // (x - mean(x)) * rsqrt(mean((x - mean(x))^2) + eps)
  int d, rstd;
  if (!t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is(q, COMFUSE_OP_RSQRT); }, d, rstd)) return false;
  t.use(k); t.use(rstd);
  int var, epsn;
  if (!t.split(t.nd(rstd).in0, COMFUSE_OP_ADD, [&](int q) { return t.is_const(q); }, var, epsn)) return false;
  t.use(t.nd(rstd).in0);
  m.eps = an.cval[epsn];
  if (!t.is(var, COMFUSE_OP_RED_MEAN)) return false;
  t.use(var);
  const int sq = t.nd(var).in0;
  const bool squared = t.is(sq, COMFUSE_OP_SQUARE) ? t.nd(sq).in0 == d : (t.is(sq, COMFUSE_OP_MUL) && t.nd(sq).in0 == d && t.nd(sq).in1 == d);
  if (!squared) return false;
  t.use(sq);
  if (!t.is(d, COMFUSE_OP_SUB)) return false;
  t.use(d);
  const int x = t.nd(d).in0, mean = t.nd(d).in1;
  if (!t.is(mean, COMFUSE_OP_RED_MEAN) || t.nd(mean).in0 != x) return false;
  t.use(mean);
  bool had_act;
  if (!t.entry(x, false, m, had_act)) return false;
  if (!t.all_live_used()) return false;
  m.kind = COMFUSE_EPI_BIAS_RES_LAYERNORM;
  return m.eps >= 0.f;
}

bool match_rmsnorm(const Analysis& an, FusedMatch& m) {
  Matcher t(an);
  int k = an.terminal, other, hit;
  const int y = k;
  if (t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is(q, COMFUSE_OP_ROWVEC); }, other, hit)) {
    m.gamma = t.nd(hit).param; t.use(k); t.use(hit); k = other;
  }
  int x, rstd;
  if (!t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is(q, COMFUSE_OP_RSQRT); }, x, rstd)) return false;
  t.use(k); t.use(rstd);
  int ms, epsn;
  if (!t.split(t.nd(rstd).in0, COMFUSE_OP_ADD, [&](int q) { return t.is_const(q); }, ms, epsn)) return false;
  t.use(t.nd(rstd).in0);
  m.eps = an.cval[epsn];
  if (!t.is(ms, COMFUSE_OP_RED_MEAN)) return false;
  t.use(ms);
  const int sq = t.nd(ms).in0;
  const bool squared = t.is(sq, COMFUSE_OP_SQUARE) ? t.nd(sq).in0 == x : (t.is(sq, COMFUSE_OP_MUL) && t.nd(sq).in0 == x && t.nd(sq).in1 == x);
  if (!squared) return false;
  t.use(sq);
  bool had_act;
  if (!t.entry(x, true, m, had_act)) return false;
  if (had_act ? !gelu_entry_order_ok(an, x) : false) return false;
  if (!had_act) m.flags |= COMFUSE_FLAG_NO_ACTIVATION;
  // the chained second reduction: row outputs may be the max and/or the arg max of Y
  for (size_t r = 0; r < an.row_outputs.size(); ++r) {
    const int q = an.row_outputs[r];
    if (t.is(q, COMFUSE_OP_RED_MAX) && t.nd(q).in0 == y && m.row_max_out < 0) { m.row_max_out = static_cast<int>(r); t.use(q); }
    else if (t.is(q, COMFUSE_OP_RED_ARGMAX) && t.nd(q).in0 == y && m.row_argmax_out < 0) { m.row_argmax_out = static_cast<int>(r); t.use(q); }
    else return false;
  }
  if (!t.all_live_used()) return false;
  m.kind = COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX;
  return m.eps >= 0.f;
}

bool match_softmax(const Analysis& an, FusedMatch& m) {
  if (!an.row_outputs.empty()) return false;
  Matcher t(an);
  const int k = an.terminal;
  int e, sum;
  if (t.is(k, COMFUSE_OP_DIV)) {
    e = t.nd(k).in0; sum = t.nd(k).in1;
  } else {
    int rc;
    if (!t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is(q, COMFUSE_OP_RECIP); }, e, rc)) return false;
    t.use(rc);
    sum = t.nd(rc).in0;
  }
  t.use(k);
  if (!t.is(sum, COMFUSE_OP_RED_SUM) || t.nd(sum).in0 != e || !t.is(e, COMFUSE_OP_EXP)) return false;
  t.use(sum); t.use(e);
  const int d = t.nd(e).in0;
  if (!t.is(d, COMFUSE_OP_SUB)) return false;
  t.use(d);
  int s = t.nd(d).in0;
  const int mx = t.nd(d).in1;
  if (!t.is(mx, COMFUSE_OP_RED_MAX) || t.nd(mx).in0 != s) return false;
  t.use(mx);
  int other, hit;
  if (t.split(s, COMFUSE_OP_ADD, [&](int q) { return t.is(q, COMFUSE_OP_CAUSAL_MASK); }, other, hit)) {
    m.causal = 1; t.use(s); t.use(hit); s = other;
  }
  // soft-cap: c2 * tanh(c1 * u) with c1 * c2 = 1
  int th, c2;
  if (t.split(s, COMFUSE_OP_MUL, [&](int q) { return t.is_const(q); }, th, c2) && t.is(th, COMFUSE_OP_TANH)) {
    int u, c1;
    if (!t.split(t.nd(th).in0, COMFUSE_OP_MUL, [&](int q) { return t.is_const(q); }, u, c1)) return false;
    const float cap = an.cval[c2];
    if (!(cap > 0.f) || std::fabs(an.cval[c1] * cap - 1.f) > 1e-5f) return false;
    m.softcap = cap;
    t.use(s); t.use(th); t.use(t.nd(th).in0);
    s = u;
  }
  if (t.split(s, COMFUSE_OP_MUL, [&](int q) { return t.is_const(q); }, other, hit)) {
    m.alpha = an.cval[hit]; t.use(s); s = other;
  }
  if (!t.is(s, COMFUSE_OP_ACC)) return false;
  t.use(s);
  if (!t.all_live_used()) return false;
  m.kind = COMFUSE_EPI_SCALE_MASK_SOFTMAX;
  return true;
}

// act(alpha * acc + bias) with nothing else alive: no reduction, no row output
bool match_elementwise(const Analysis& an, FusedMatch& m) {
  if (!an.row_outputs.empty() || an.n_reductions != 0) return false;
  Matcher t(an);
  int k = an.terminal, other, hit;
  for (int op : {COMFUSE_OP_RELU, COMFUSE_OP_GELU_TANH, COMFUSE_OP_TANH, COMFUSE_OP_SIGMOID})
    if (m.activation == 0 && t.is(k, op)) { m.activation = op; t.use(k); k = t.nd(k).in0; }
  if (t.split(k, COMFUSE_OP_ADD, [&](int q) { return t.is(q, COMFUSE_OP_ROWVEC); }, other, hit)) {
    m.bias = t.nd(hit).param; t.use(k); t.use(hit); k = other;
  }
  if (t.split(k, COMFUSE_OP_MUL, [&](int q) { return t.is_const(q); }, other, hit)) {
    m.alpha = an.cval[hit]; t.use(k); k = other;
  }
  if (!t.is(k, COMFUSE_OP_ACC)) return false;
  t.use(k);
  if (!t.all_live_used()) return false;
  m.kind = COMFUSE_EPI_BIAS_ACTIVATION;
  return true;
}

bool match_fused(const Analysis& an, FusedMatch& m) {
  { FusedMatch t; if (match_elementwise(an, t)) { m = t; return true; } }
  { FusedMatch t; if (match_layernorm(an, t)) { m = t; return true; } }
  { FusedMatch t; if (match_rmsnorm(an, t)) { m = t; return true; } }
  { FusedMatch t; if (match_softmax(an, t)) { m = t; return true; } }
  return false;
}

// ------------------------------------------------------------------------------------------------ stage program
// Lowering for the on-chip interpreter (fused_params.h: StageProgram): possible when ONE tensor stays resident
// across the stage boundaries (Sec. 5.3: the reduction's statistics and the passed-through original tensor are the
// two entry points of the nested sub-program) and every tensor-valued expression is a chain on it.
struct StageBinding {
  int rowvec_param[3] = {-1, -1, -1};
  int n_rowvec = 0;
  int tensor_param = -1;
  int row_out_pos[kStageMaxRowOut] = {};  // StageProgram::out[r] is row output number row_out_pos[r]
};

struct StageLowering {
  const Analysis& an;
  StageBinding& bind;
  std::vector<int> scalar_of;  // per node: its per-row scalar index, -1 = none
  std::vector<int> recip_of;   // per node: the scalar holding its reciprocal, -1 = not needed yet
  int x_root = -1;
  bool pass0 = false;          // the code being emitted runs in pass 0 (the full-tensor operand is at hand there)
  int temps_in_use = 0;        // temporaries holding a value at this point of the code being emitted
  bool uses_temps = false;
  int scalars = 0;             // per-row scalars allocated so far
  StageProgram* sp = nullptr;
  explicit StageLowering(const Analysis& a, StageBinding& b) : an(a), bind(b), scalar_of(a.n, -1), recip_of(a.n, -1) {}

  // v / s with s a per-row value (or constant) becomes v * (1 / s): one reciprocal per row instead of one per element
  bool divide_by(int k, ChainInstr& ci) {
    if (ci.operand == CHO_CONST) { ci.op = COMFUSE_OP_MUL; ci.imm = 1.f / ci.imm; return true; }
    if (ci.operand != CHO_SCALAR) { ci.op = COMFUSE_OP_DIV; return true; }
    if (recip_of[k] < 0) {
      if (scalars >= kStageMaxScalars || sp->n_scalar_instr >= kStageMaxScalarInstr || an.stage[k] < 1) return false;
      ScalarInstr& si = sp->sc[sp->n_scalar_instr++];
      si.after_pass = static_cast<uint8_t>(an.stage[k] - 1);
      si.op = COMFUSE_OP_RECIP;
      si.dst = static_cast<uint8_t>(scalars);
      si.a_kind = CHO_SCALAR; si.a = static_cast<uint8_t>(scalar_of[k]); si.a_imm = 0.f;
      si.b_kind = CHO_CONST; si.b = 0; si.b_imm = 0.f;
      recip_of[k] = scalars++;
    }
    ci.op = COMFUSE_OP_MUL;
    ci.index = static_cast<int16_t>(recip_of[k]);
    return true;
  }

  bool tensor(int k) const { return an.type[k] == T_TENSOR; }
  // can node k be the right-hand operand of a chain instruction?
  bool operand(int k, bool entry_mode, ChainInstr& ci) {
    ci.operand = CHO_NONE; ci.index = 0; ci.imm = 0.f;
    if (an.type[k] == T_CONST) { ci.operand = CHO_CONST; ci.imm = an.cval[k]; return true; }
    if (an.type[k] == T_ROW) {
      if (scalar_of[k] < 0) return false;
      ci.operand = CHO_SCALAR; ci.index = static_cast<int16_t>(scalar_of[k]);
      return true;
    }
    switch (an.nodes[k].op) {
      case COMFUSE_OP_ROWVEC: {
        const int q = an.nodes[k].param;
        int slot = -1;
        for (int i = 0; i < bind.n_rowvec; ++i) if (bind.rowvec_param[i] == q) slot = i;
        if (slot < 0) {
          if (bind.n_rowvec == 3) return false;
          slot = bind.n_rowvec++;
          bind.rowvec_param[slot] = q;
        }
        ci.operand = CHO_ROWVEC; ci.index = static_cast<int16_t>(slot);
        return true;
      }
      case COMFUSE_OP_TENSOR:
        if (!entry_mode && !pass0) return false;  // the operand ring delivers it once, in pass 0
        if (bind.tensor_param >= 0 && bind.tensor_param != an.nodes[k].param) return false;
        bind.tensor_param = an.nodes[k].param;
        ci.operand = CHO_RESIDUAL;
        return true;
      case COMFUSE_OP_CAUSAL_MASK: ci.operand = CHO_MASK; return true;
      default: return false;
    }
  }
  bool is_root(int k, bool entry_mode) const { return entry_mode ? an.nodes[k].op == COMFUSE_OP_ACC : k == x_root; }
  // code that turns the root's value into node k's value (v holds the root's value where the code starts)
  bool chain(int k, bool entry_mode, std::vector<ChainInstr>& out, bool in_pass0 = false) {
    bool v_root = true;
    pass0 = entry_mode || in_pass0;
    return emit(k, entry_mode, out, v_root);
  }
  // code that leaves node k's value in v; `v_root`: v holds the root's value at this point
  bool emit(int k, bool entry_mode, std::vector<ChainInstr>& out, bool& v_root) {
    const size_t mark = out.size();
    const bool v_root_in = v_root;
    const int temps_in = temps_in_use;
    if (emit_node(k, entry_mode, out, v_root)) return true;
    out.resize(mark);  // a failed attempt leaves no code behind
    v_root = v_root_in;
    temps_in_use = temps_in;
    return false;
  }
  bool emit_node(int k, bool entry_mode, std::vector<ChainInstr>& out, bool& v_root) {
    if (is_root(k, entry_mode)) {
      if (!v_root) out.push_back(ChainInstr{static_cast<uint8_t>(kChainXload), CHO_NONE, 0, 0.f});  // x: the root (before XSAVE: the accumulator)
      v_root = true;
      return true;
    }
    if (!tensor(k)) return false;
    const comfuse_spec_node_t& nd = an.nodes[k];
    if (is_unary(nd.op)) {
      if (!emit(nd.in0, entry_mode, out, v_root)) return false;
      v_root = false;
      out.push_back(ChainInstr{static_cast<uint8_t>(nd.op), CHO_NONE, 0, 0.f});
      return true;
    }
    ChainInstr ci;
    if (is_leaf(nd.op)) {
      // a chain that starts from a broadcast (row vector, causal mask, in pass 0 the full tensor): v = operand
      if (!operand(k, entry_mode, ci)) return false;
      ci.op = static_cast<uint8_t>(kChainMov);
      out.push_back(ci);
      v_root = false;
      return true;
    }
    if (!is_binary(nd.op)) return false;
    const int a = nd.in0, b = nd.in1;
    auto carrier = [&](int q) { return is_root(q, entry_mode) || (tensor(q) && !is_leaf(an.nodes[q].op)); };
    if (a == b && nd.op == COMFUSE_OP_MUL && carrier(a)) {
      if (!emit(a, entry_mode, out, v_root)) return false;
      out.push_back(ChainInstr{COMFUSE_OP_SQUARE, CHO_NONE, 0, 0.f});
      v_root = false;
      return true;
    }
    auto starts = [&](int q) { return carrier(q) || (tensor(q) && is_leaf(an.nodes[q].op)); };  // something a chain can begin with
    if (starts(a) && !carrier(b) && operand(b, entry_mode, ci)) {
      if (!emit(a, entry_mode, out, v_root)) return false;
      ci.op = static_cast<uint8_t>(nd.op);
      if (nd.op == COMFUSE_OP_DIV && !divide_by(b, ci)) return false;
      out.push_back(ci);
      v_root = false;
      return true;
    }
    if (starts(b) && !carrier(a) && operand(a, entry_mode, ci)) {
      if (!emit(b, entry_mode, out, v_root)) return false;
      ci.op = static_cast<uint8_t>(nd.op == COMFUSE_OP_SUB ? kChainRsub : nd.op == COMFUSE_OP_DIV ? kChainRdiv : nd.op);
      out.push_back(ci);
      v_root = false;
      return true;
    }
    // a computed tensor combined with the root itself (a gate: x * sigmoid(x)): the root is at hand in every pass
    if (is_root(a, entry_mode) && carrier(b) && !is_root(b, entry_mode)) {
      if (!emit(b, entry_mode, out, v_root)) return false;
      out.push_back(ChainInstr{static_cast<uint8_t>(nd.op == COMFUSE_OP_SUB ? kChainRsub : nd.op == COMFUSE_OP_DIV ? kChainRdiv : nd.op),
                               CHO_X, 0, 0.f});
      v_root = false;
      return true;
    }
    if (is_root(b, entry_mode) && carrier(a) && !is_root(a, entry_mode)) {
      if (!emit(a, entry_mode, out, v_root)) return false;
      out.push_back(ChainInstr{static_cast<uint8_t>(nd.op), CHO_X, 0, 0.f});
      v_root = false;
      return true;
    }
    // two computed tensors meet: the first goes into a temporary while the second is computed (generated kernels only: the
    // temporaries are registers of straight-line code there; shared sub-expressions are the compiler's to find)
    if (carrier(a) && carrier(b) && temps_in_use < kStageMaxTemps) {
      if (!emit(a, entry_mode, out, v_root)) return false;
      const int t = temps_in_use++;
      out.push_back(ChainInstr{static_cast<uint8_t>(kChainTsave), CHO_NONE, static_cast<int16_t>(t), 0.f});
      if (!emit(b, entry_mode, out, v_root)) return false;
      // v = b, temporary = a: a (op) b in the reversed forms where the order matters
      out.push_back(ChainInstr{static_cast<uint8_t>(nd.op == COMFUSE_OP_SUB ? kChainRsub : nd.op == COMFUSE_OP_DIV ? kChainRdiv : nd.op),
                               CHO_T, static_cast<int16_t>(t), 0.f});
      --temps_in_use;
      uses_temps = true;
      v_root = false;
      return true;
    }
    return false;  // more live tensors than temporaries, or two broadcasts
  }
};

bool lower_stage_program_from(const Analysis& an, int x_root, StageProgram& sp, StageBinding& bind);

bool lower_stage_program(const Analysis& an, StageProgram& sp, StageBinding& bind) {
  if (!an.row_outputs.empty() && an.row_outputs.size() > static_cast<size_t>(kStageMaxRowOut)) return false;
  if (an.type[an.terminal] != T_TENSOR) return false;
  const int n = an.n;
  // the resident tensor: the one stage-0 tensor that later stages read
  std::vector<int> cand;
  for (int k = 0; k < n; ++k) {
    if (!an.live[k]) continue;
    if (an.type[k] != T_TENSOR || an.stage[k] < 1 || is_reduce(an.nodes[k].op)) continue;
    for (int e : {an.nodes[k].in0, an.nodes[k].in1}) {
      if (e < 0 || an.type[e] != T_TENSOR || an.stage[e] != 0) continue;
      const int eop = an.nodes[e].op;
      if (is_leaf(eop) && eop != COMFUSE_OP_ACC) continue;  // broadcasts are re-read, not resident
      bool seen = false;
      for (int c : cand) seen |= c == e;
      if (!seen) cand.push_back(e);
    }
  }
  // (several such tensors: none of them can be THE resident one, but a tensor below them all -- in the end the accumulator
  // itself -- can, with the others recomputed from it in every pass that reads them: the loop below)
  if (cand.size() == 1) {
    StageBinding b1;
    if (lower_stage_program_from(an, cand[0], sp, b1)) { bind = b1; return true; }
  }
  // no later stage reads a stage-0 tensor (the reductions only feed row outputs), or the one they read is not a chain on
  // the accumulator (a gate x * f(x)): any stage-0 tensor from which the terminal, every reduction input and every tensor
  // the later stages read can be reached by chains will do; try them from the last to the first
  for (int k = n - 1; k >= 0; --k) {
    if (!an.live[k] || an.type[k] != T_TENSOR || an.stage[k] != 0) continue;
    if (is_leaf(an.nodes[k].op) && an.nodes[k].op != COMFUSE_OP_ACC) continue;
    StageBinding b2;
    if (lower_stage_program_from(an, k, sp, b2)) { bind = b2; return true; }
  }
  return false;
}

bool lower_stage_program_from(const Analysis& an, int x_root, StageProgram& sp, StageBinding& bind) {
  std::memset(&sp, 0, sizeof(sp));
  StageLowering L(an, bind);
  L.sp = &sp;
  L.x_root = x_root;
  const int n = an.n;
  // stage 0: acc -> x
  std::vector<ChainInstr> entry, fin;
  std::vector<std::vector<ChainInstr>> red_chain;
  if (!L.chain(L.x_root, true, entry)) return false;
  // reductions and per-row arithmetic, in node order
  int max_pass = an.stage[an.terminal];
  int& scalars = L.scalars;
  int topk_input[kStageMaxRed];        // per reduction: the input node of a Top-K, else -1
  std::vector<int> topk_of(n, -1);     // per Top-K node: its reduction
  for (int r = 0; r < kStageMaxRed; ++r) topk_input[r] = -1;
  for (int k = 0; k < n; ++k) {
    if (!an.live[k] || an.type[k] != T_ROW) continue;
    const comfuse_spec_node_t& nd = an.nodes[k];
    if (is_topk(nd.op)) {
      // values and columns of the same input and K share one reduction; on chip K <= kStageMaxTopK
      const int e = nd.in0;
      if (nd.param > kStageMaxTopK || an.type[e] != T_TENSOR) return false;
      int found = -1;
      for (int r = 0; r < sp.n_red; ++r)
        if (sp.red[r].k == nd.param && topk_input[r] == e) found = r;
      if (found < 0) {
        if (sp.n_red >= kStageMaxRed) return false;
        StageReduction& r = sp.red[sp.n_red];
        r.op = COMFUSE_OP_RED_ARGMAX;
        r.k = static_cast<uint8_t>(nd.param);
        r.pass = static_cast<uint8_t>(an.stage[e]);
        red_chain.emplace_back();
        if (e == an.terminal) r.on_terminal = 1;
        else if (!L.chain(e, false, red_chain.back())) return false;  // (no full tensor: the later rounds re-run this code)
        if (r.pass > max_pass) max_pass = r.pass;
        topk_input[sp.n_red] = e;
        found = sp.n_red++;
      }
      topk_of[k] = found;
      continue;
    }
    if (scalars >= kStageMaxScalars) return false;
    const int my = scalars++;  // before the chains below, which may allocate reciprocals
    if (is_reduce(nd.op)) {
      if (sp.n_red >= kStageMaxRed) return false;
      const int e = nd.in0;
      if (an.type[e] != T_TENSOR) return false;
      StageReduction& r = sp.red[sp.n_red];
      r.op = static_cast<uint8_t>(nd.op);
      r.pass = static_cast<uint8_t>(an.stage[e]);
      r.dst = static_cast<uint8_t>(my);
      red_chain.emplace_back();
      if (e == an.terminal) r.on_terminal = 1;
      else if (!L.chain(e, false, red_chain.back(), r.pass == 0)) return false;
      if (r.pass > max_pass) max_pass = r.pass;
      ++sp.n_red;
    } else {
      if (sp.n_scalar_instr >= kStageMaxScalarInstr || an.stage[k] < 1) return false;
      ScalarInstr& si = sp.sc[sp.n_scalar_instr++];
      si.after_pass = static_cast<uint8_t>(an.stage[k] - 1);
      si.op = static_cast<uint8_t>(nd.op);
      si.dst = static_cast<uint8_t>(my);
      auto set = [&](int e, uint8_t& kind, uint8_t& ix, float& imm) {
        if (e < 0) { kind = CHO_CONST; ix = 0; imm = 0.f; return true; }
        if (an.type[e] == T_CONST) { kind = CHO_CONST; ix = 0; imm = an.cval[e]; return true; }
        if (an.type[e] != T_ROW || L.scalar_of[e] < 0) return false;
        kind = CHO_SCALAR; ix = static_cast<uint8_t>(L.scalar_of[e]); imm = 0.f;
        return true;
      };
      if (!set(nd.in0, si.a_kind, si.a, si.a_imm) || !set(nd.in1, si.b_kind, si.b, si.b_imm)) return false;
    }
    L.scalar_of[k] = my;
  }
  // the terminal: x -> y
  if (!L.chain(an.terminal, false, fin, an.stage[an.terminal] == 0)) return false;
  sp.terminal_pass = static_cast<uint8_t>(an.stage[an.terminal]);
  if (max_pass + 1 > kStageMaxPasses) return false;
  sp.n_passes = static_cast<uint8_t>(max_pass + 1);
  // a reduction on y is accumulated in the terminal's pass
  for (int r = 0; r < sp.n_red; ++r)
    if (sp.red[r].on_terminal) sp.red[r].pass = sp.terminal_pass;
  // the micro-instruction stream of every pass
  int nc = 0;
  bool ok = true;
  auto emit = [&](ChainInstr c) { if (nc < kStageMaxCode) sp.code[nc++] = c; else ok = false; };
  auto micro = [&](int op, int index = 0) { emit(ChainInstr{static_cast<uint8_t>(op), CHO_NONE, static_cast<int16_t>(index), 0.f}); };
  for (int pass = 0; pass < sp.n_passes; ++pass) {
    sp.pass_off[pass] = static_cast<uint8_t>(nc);
    bool v_is_x = true;  // at the start of a later pass v = x as loaded from TMEM
    if (pass == 0) {
      for (const ChainInstr& c : entry) emit(c);
      micro(kChainXsave);
    }
    for (int r = 0; r < sp.n_red; ++r) {
      if (sp.red[r].pass != pass || sp.red[r].on_terminal) continue;
      sp.red[r].code_lo = static_cast<uint8_t>(nc);  // from here (v = x, reloaded if it was changed) to the ACC
      if (!v_is_x) micro(kChainXload);
      for (const ChainInstr& c : red_chain[r]) emit(c);
      v_is_x = red_chain[r].empty();
      micro(kChainAcc, r);
      sp.red[r].code_hi = static_cast<uint8_t>(nc);
    }
    if (pass == sp.terminal_pass) {
      const int fin_lo = nc;
      if (!v_is_x) micro(kChainXload);
      for (const ChainInstr& c : fin) emit(c);
      for (int r = 0; r < sp.n_red; ++r)
        if (sp.red[r].on_terminal) {
          micro(kChainAcc, r);
          sp.red[r].code_lo = static_cast<uint8_t>(fin_lo);
          sp.red[r].code_hi = static_cast<uint8_t>(nc);
        }
      micro(kChainEmit);
    }
  }
  sp.pass_off[sp.n_passes] = static_cast<uint8_t>(nc);
  if (!ok) return false;
  for (size_t r = 0; r < an.row_outputs.size(); ++r) {
    const int q = an.row_outputs[r];
    if (is_topk(an.nodes[q].op)) {
      if (topk_of[q] < 0) return false;
      sp.out[r].topk_red = static_cast<uint8_t>(topk_of[q] + 1);
      sp.out[r].is_int = an.nodes[q].op == COMFUSE_OP_RED_TOPK_INDICES;
      sp.x_writeback = 1;
      bind.row_out_pos[r] = static_cast<int>(r);
      continue;
    }
    if (an.type[q] != T_ROW || L.scalar_of[q] < 0) return false;
    sp.out[r].scalar = static_cast<uint8_t>(L.scalar_of[q]);
    sp.out[r].is_int = an.nodes[q].op == COMFUSE_OP_RED_ARGMAX;
    bind.row_out_pos[r] = static_cast<int>(r);
  }
  // a Top-K that no row output takes would still be swept K times: drop it back to a plain arg max
  for (int r = 0; r < sp.n_red; ++r) {
    bool used = false;
    for (size_t o = 0; o < an.row_outputs.size(); ++o) used |= sp.out[o].topk_red == r + 1;
    if (!used) sp.red[r].k = 0;
  }
  sp.n_row_out = static_cast<uint8_t>(an.row_outputs.size());
  // the sweep table: each pass, then the further rounds of that pass's Top-K reductions in program order
  int ns = 0;
  for (int pass = 0; pass < sp.n_passes; ++pass) {
    sp.sweep[ns++] = SweepStep{sp.pass_off[pass], sp.pass_off[pass + 1], -1, 0, static_cast<uint8_t>(pass), 0, {0, 0}};
    for (int r = 0; r < sp.n_red; ++r) {
      if (sp.red[r].pass != pass) continue;
      for (int round = 1; round < sp.red[r].k; ++round)
        sp.sweep[ns++] = SweepStep{sp.red[r].code_lo, sp.red[r].code_hi, static_cast<int8_t>(r), static_cast<uint8_t>(round),
                                   static_cast<uint8_t>(pass), 0, {0, 0}};
    }
  }
  sp.sweep[ns - 1].release = 1;
  sp.n_sweeps = static_cast<uint8_t>(ns);
  sp.uses_temps = L.uses_temps ? 1 : 0;
  return true;
}

// ------------------------------------------------------------------------------------------------ row program
comfuse_status_t lower_row_program(const Analysis& an, int N, RowProgram& P, int& n_instr, int& n_slots) {
  const int n = an.n;
  std::vector<int> last_use(n, -1);
  for (int k = 0; k < n; ++k) {
    if (!an.live[k] || an.type[k] == T_CONST) continue;
    if (an.nodes[k].in0 >= 0) last_use[an.nodes[k].in0] = k;
    if (an.nodes[k].in1 >= 0) last_use[an.nodes[k].in1] = k;
  }
  last_use[an.terminal] = n;
  for (int r : an.row_outputs) last_use[r] = n;
  std::vector<Operand> ref(n, Operand{OPK_NONE, 0, 0, 0.f});
  std::vector<int> free_slots;
  int slots = 0, scalars = 0, ni = 0;
  for (int k = 0; k < n; ++k) {
    if (!an.live[k]) continue;
    const comfuse_spec_node_t& nd = an.nodes[k];
    if (an.type[k] == T_CONST) { ref[k] = Operand{OPK_CONST, 0, 0, an.cval[k]}; continue; }
    switch (nd.op) {
      case COMFUSE_OP_ACC: ref[k] = Operand{OPK_ACC, 0, 0, 0.f}; continue;
      case COMFUSE_OP_ROWVEC: ref[k] = Operand{OPK_ROWVEC, 0, static_cast<int16_t>(nd.param), 0.f}; continue;
      case COMFUSE_OP_TENSOR: ref[k] = Operand{OPK_TENSOR, 0, static_cast<int16_t>(nd.param), 0.f}; continue;
      case COMFUSE_OP_CAUSAL_MASK: ref[k] = Operand{OPK_MASK, 0, 0, 0.f}; continue;
      default: break;
    }
    if (ni >= kRowMaxInstr) return COMFUSE_ERR_UNSUPPORTED;
    RowInstr& in = P.ins[ni++];
    in.op = static_cast<uint8_t>(nd.op);
    in.a = ref[nd.in0];
    in.b = nd.in1 >= 0 ? ref[nd.in1] : Operand{OPK_NONE, 0, 0, 0.f};
    if (is_topk(nd.op)) {
      // written straight to its row output, K values per row: dst = position in the row-output list, b.index = K
      if (nd.param > N) return COMFUSE_ERR_INVALID_ARG;
      int pos = -1;
      for (size_t r = 0; r < an.row_outputs.size(); ++r)
        if (an.row_outputs[r] == k) { pos = static_cast<int>(r); break; }
      in.dst_scalar = 1;
      in.dst = static_cast<int16_t>(pos);
      in.b = Operand{OPK_NONE, 0, static_cast<int16_t>(nd.param), 0.f};
      ref[k] = Operand{OPK_NONE, 0, 0, 0.f};
    } else if (an.type[k] == T_ROW) {
      if (scalars >= kRowMaxScalars) return COMFUSE_ERR_UNSUPPORTED;
      in.dst_scalar = 1;
      in.dst = static_cast<int16_t>(scalars);
      ref[k] = Operand{OPK_SCALAR, 0, static_cast<int16_t>(scalars), 0.f};
      ++scalars;
    } else {
      in.dst_scalar = 0;
      // overwrite an operand's buffer in place if this is its last use, else take a free buffer, else a new one
      int slot = -1;
      for (int e : {nd.in0, nd.in1})
        if (slot < 0 && e >= 0 && ref[e].kind == OPK_SLOT && last_use[e] == k) slot = ref[e].index;
      if (slot < 0) {
        if (!free_slots.empty()) { slot = free_slots.back(); free_slots.pop_back(); }
        else slot = slots++;
      }
      in.dst = static_cast<int16_t>(slot);
      ref[k] = Operand{OPK_SLOT, 0, static_cast<int16_t>(slot), 0.f};
    }
    // release the buffers whose last reader this was (unless just taken over)
    for (int e : {nd.in0, nd.in1}) {
      if (e < 0 || ref[e].kind != OPK_SLOT || last_use[e] != k) continue;
      if (ref[k].kind == OPK_SLOT && ref[k].index == ref[e].index) continue;
      bool already = false;
      for (int f : free_slots) already |= f == ref[e].index;
      if (!already) free_slots.push_back(ref[e].index);
    }
  }
  if (static_cast<size_t>(slots) * N * sizeof(float) > kRowMaxSlotBytes) return COMFUSE_ERR_UNSUPPORTED;
  P.terminal = ref[an.terminal];
  P.n_row_out = static_cast<int>(an.row_outputs.size());
  for (int r = 0; r < P.n_row_out; ++r) {
    P.row_out_src[r] = ref[an.row_outputs[r]];
    P.row_out_int[r] = an.nodes[an.row_outputs[r]].op == COMFUSE_OP_RED_ARGMAX && an.type[an.row_outputs[r]] == T_ROW;
  }
  P.n_instr = ni;
  P.n_slots = slots;
  n_instr = ni;
  n_slots = slots;
  return COMFUSE_OK;
}

comfuse_status_t validate_shape(const comfuse_gemm_shape_t* s) {
  if (!s) return COMFUSE_ERR_INVALID_ARG;
  if (s->batch < 1 || s->M < 1 || s->N < 1 || s->K < 1) return COMFUSE_ERR_INVALID_ARG;
  if (s->flags & ~COMFUSE_FLAG_B_ROW_MAJOR_NK) return COMFUSE_ERR_INVALID_ARG;
  const bool b_nk = (s->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0;
  if (s->lda < s->K || s->ldb < (b_nk ? s->K : s->N) || s->ldy < s->N) return COMFUSE_ERR_INVALID_ARG;
  if ((s->N & 7) || (s->K & 7) || (s->lda & 7) || (s->ldb & 7) || (s->ldy & 7)) return COMFUSE_ERR_ALIGNMENT;
  if (s->batch > 1) {
    if (s->batch_stride_a < static_cast<long long>(s->M - 1) * s->lda + s->K) return COMFUSE_ERR_INVALID_ARG;
    if (s->batch_stride_b < (b_nk ? static_cast<long long>(s->N - 1) * s->ldb + s->K : static_cast<long long>(s->K - 1) * s->ldb + s->N))
      return COMFUSE_ERR_INVALID_ARG;
    if (s->batch_stride_y < static_cast<long long>(s->M - 1) * s->ldy + s->N) return COMFUSE_ERR_INVALID_ARG;
    if ((s->batch_stride_a & 7) || (s->batch_stride_b & 7) || (s->batch_stride_y & 7)) return COMFUSE_ERR_ALIGNMENT;
  }
  return COMFUSE_OK;
}

// The descriptor of the fused instantiation a matched program lowers to.
comfuse_gemm_desc_t fused_desc(const comfuse_gemm_shape_t& s, const FusedMatch& m, long long ldr) {
  comfuse_gemm_desc_t d;
  std::memset(&d, 0, sizeof(d));
  d.batch = s.batch; d.M = s.M; d.N = s.N; d.K = s.K;
  d.lda = s.lda; d.ldb = s.ldb; d.ldy = s.ldy; d.ldr = ldr;
  d.batch_stride_a = s.batch_stride_a; d.batch_stride_b = s.batch_stride_b; d.batch_stride_y = s.batch_stride_y;
  d.batch_stride_r = static_cast<long long>(s.M) * ldr;
  d.kind = m.kind;
  d.mask = m.causal ? COMFUSE_MASK_CAUSAL : COMFUSE_MASK_NONE;
  d.alpha = m.alpha; d.eps = m.eps; d.fused = 1; d.flags = m.flags | (s.flags & COMFUSE_FLAG_B_ROW_MAJOR_NK); d.softcap = m.softcap;
  return d;
}

// Which interpreter for a program both can run?  Both cost roughly a fixed time per element and executed instruction
// (measured on four programs on one B200: about 0.36 ns per micro-instruction on-chip -- 8 epilogue warps per SM, the
// chains re-run in every pass, transcendental operations counted three times -- against 0.9 ns per instruction plus 0.6 ns for
// the bf16 round trip of Z in the row program, which has every SM's full occupancy).  A coarse model, good enough to send
// exponential-heavy three-pass programs to the row program and the rest on-chip.
// Whether `fused` = 1 runs an on-chip program as a kernel generated for it: where the run-time compiler is there, unless
// COMFUSE_GENERATE=0 asks for the interpreter.
bool generate_by_default() {
  const char* v = std::getenv("COMFUSE_GENERATE");
  if (v && v[0] == '0') return false;
  return program_compiler_status(nullptr) == COMFUSE_OK;
}

bool on_chip_is_cheaper(const Analysis& an, const StageProgram& sp, int N) {
  RowProgram P;
  std::memset(&P, 0, sizeof(P));
  int ni = 0, ns = 0;
  if (lower_row_program(an, N, P, ni, ns) != COMFUSE_OK) return true;  // the row program cannot run it at all
  float units = 0.f;
  for (int pass = 0; pass < sp.n_passes; ++pass) {
    units += 2.f;  // fragment load, loop overhead
    for (int i = sp.pass_off[pass]; i < sp.pass_off[pass + 1]; ++i) {
      const int op = sp.code[i].op;
      const bool transcendental = op == COMFUSE_OP_EXP || op == COMFUSE_OP_LOG || op == COMFUSE_OP_TANH || op == COMFUSE_OP_GELU_TANH ||
                                  op == COMFUSE_OP_SIGMOID || op == COMFUSE_OP_DIV || op == kChainRdiv || op == COMFUSE_OP_RECIP;
      units += transcendental ? 3.f : 1.f;
    }
  }
  // compiled into the kernel, the same stream costs about 0.14 ns per unit (measured on the same programs: 2.2 to 2.8 times
  // the interpreter's rate)
  return (generate_by_default() ? 0.14f : 0.36f) * units <= 0.9f * static_cast<float>(ni) + 0.6f;
}

struct Decision {
  Analysis an;
  FusedMatch match;
  bool fused = false;       // a compiled fused kind
  bool on_chip = false;     // the on-chip stage program (generated kernel or interpreter)
  bool interp_ok = false;   // ... which the interpreter can run (no temporaries)
  StageProgram stage_prog;
  StageBinding stage_bind;
  size_t fused_inner_ws = 0;  // what the fused entry point itself needs
  size_t fused_scratch = 0;   // row max / arg max the caller did not ask for
};

comfuse_status_t decide(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, int want_fused, Decision& dc) {
  comfuse_status_t s = validate_shape(shape);
  if (s != COMFUSE_OK) return s;
  s = analyse(spec, dc.an);
  if (s != COMFUSE_OK) return s;
  if (want_fused == 1 && match_fused(dc.an, dc.match)) {
    const comfuse_gemm_desc_t d = fused_desc(*shape, dc.match, shape->N);
    size_t ws = 0;
    if (dc.match.kind == COMFUSE_EPI_BIAS_ACTIVATION) {
      dc.fused = true;  // the plain GEMM's tiling takes any shape the validation let through
    } else if (comfuse_workspace_size(&d, &ws) == COMFUSE_OK) {
      dc.fused = true;
      dc.fused_inner_ws = (ws + 255) & ~static_cast<size_t>(255);
      if (dc.match.kind == COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX && (dc.match.row_max_out < 0 || dc.match.row_argmax_out < 0))
        dc.fused_scratch = 2 * static_cast<size_t>(shape->batch) * shape->M * 4;
    }
  }
  if (want_fused && !dc.fused && lower_stage_program(dc.an, dc.stage_prog, dc.stage_bind)) {
    const void* none[3] = {nullptr, nullptr, nullptr};
    auto query = [&](bool compiled) {
      return run_fused_program(shape->batch, shape->M, shape->N, shape->K, 0, 0, 0, 0, 0, 0, nullptr, nullptr, nullptr, dc.stage_prog, none,
                               nullptr, 0, nullptr, true, false, compiled) == COMFUSE_OK;
    };
    dc.interp_ok = want_fused != 3 && query(false);
    const bool generated_ok = (want_fused == 3 || (want_fused == 1 && generate_by_default())) && query(true);
    dc.on_chip = dc.interp_ok || generated_ok;
    if (dc.on_chip && want_fused == 1 && !on_chip_is_cheaper(dc.an, dc.stage_prog, shape->N)) dc.on_chip = false;
  }
  return COMFUSE_OK;
}

}  // namespace
}  // namespace comfuse

using namespace comfuse;

extern "C" {

comfuse_status_t comfuse_spec_plan(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, comfuse_spec_plan_t* plan) {
  if (!plan) return COMFUSE_ERR_INVALID_ARG;
  Decision dc;
  comfuse_status_t s = decide(spec, shape, 1, dc);
  if (s != COMFUSE_OK) return s;
  std::memset(plan, 0, sizeof(*plan));
  plan->n_stages = dc.an.n_stages;
  plan->n_reductions = dc.an.n_reductions;
  plan->n_live_nodes = dc.an.n_live;
  plan->fused_kind = -1;
  if (dc.fused) {
    plan->path = COMFUSE_SPEC_PATH_FUSED_KERNEL;
    plan->fused_kind = dc.match.kind;
    plan->fused_flags = dc.match.flags;
    plan->alpha = dc.match.alpha; plan->eps = dc.match.eps; plan->softcap = dc.match.softcap;
    plan->causal = dc.match.causal;
  }
  // what `fused` = 2 would take (the compiled kinds skipped)
  Decision d2;
  s = decide(spec, shape, 2, d2);
  if (s != COMFUSE_OK) return s;
  plan->program_path = d2.on_chip ? COMFUSE_SPEC_PATH_FUSED_PROGRAM : COMFUSE_SPEC_PATH_ROW_PROGRAM;
  if (d2.on_chip) plan->n_passes = d2.stage_prog.n_passes;
  if (!dc.fused) plan->path = dc.on_chip ? COMFUSE_SPEC_PATH_FUSED_PROGRAM : COMFUSE_SPEC_PATH_ROW_PROGRAM;
  // the row program (what `fused` = 0 runs) is described in any case
  RowProgram P;
  std::memset(&P, 0, sizeof(P));
  s = lower_row_program(dc.an, shape->N, P, plan->n_instructions, plan->n_slots);
  // where another path exists, the row program's limits are no error
  return (plan->path == COMFUSE_SPEC_PATH_ROW_PROGRAM) ? s : COMFUSE_OK;
}

comfuse_status_t comfuse_program_compiler_status(const char** why) { return program_compiler_status(why); }

comfuse_status_t comfuse_gemm_spec_prepare(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, int32_t fused) {
  if (fused < 0 || fused > 3) return COMFUSE_ERR_INVALID_ARG;
  Decision dc;
  comfuse_status_t s = decide(spec, shape, fused, dc);
  if (s != COMFUSE_OK) return s;
  if (fused == 1 && dc.on_chip && generate_by_default()) {
    (void)prepare_compiled_program(shape->N, dc.stage_prog);  // a failure leaves the interpreter
    return COMFUSE_OK;
  }
  if (fused != 3) return COMFUSE_OK;
  if (!dc.on_chip) return COMFUSE_ERR_UNSUPPORTED;
  return prepare_compiled_program(shape->N, dc.stage_prog);
}

comfuse_status_t comfuse_gemm_spec_workspace_size(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, int32_t fused,
                                                  size_t* bytes) {
  if (!bytes || fused < 0 || fused > 3) return COMFUSE_ERR_INVALID_ARG;
  Decision dc;
  comfuse_status_t s = decide(spec, shape, fused, dc);
  if (s != COMFUSE_OK) return s;
  if (fused == 3 && !dc.on_chip) return COMFUSE_ERR_UNSUPPORTED;
  if (dc.fused) {
    *bytes = dc.fused_inner_ws + dc.fused_scratch;
    return COMFUSE_OK;
  }
  if (dc.on_chip) {
    *bytes = 0;
    return COMFUSE_OK;
  }
  RowProgram P;
  std::memset(&P, 0, sizeof(P));
  int ni, ns;
  s = lower_row_program(dc.an, shape->N, P, ni, ns);
  if (s != COMFUSE_OK) return s;
  *bytes = static_cast<size_t>(shape->batch) * shape->M * shape->N * 2;
  return COMFUSE_OK;
}

comfuse_status_t comfuse_gemm_spec(const comfuse_fusion_spec_t* spec, const comfuse_gemm_shape_t* shape, const void* A, const void* B,
                                   void* Y, const void* const* params, const int64_t* param_ld, void* const* row_out, int32_t fused,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (fused < 0 || fused > 3) return COMFUSE_ERR_INVALID_ARG;
  Decision dc;
  comfuse_status_t s = decide(spec, shape, fused, dc);
  if (s != COMFUSE_OK) return s;
  if (fused == 3 && !dc.on_chip) return COMFUSE_ERR_UNSUPPORTED;  // the generated kernel is asked for by name: no other path stands in
  const bool try_generated = fused == 1 && dc.on_chip && generate_by_default();
  if (!A || !B || !Y) return COMFUSE_ERR_INVALID_ARG;
  const Analysis& an = dc.an;
  // the parameter table: every slot a live node reads must be there, aligned, with a usable leading dimension
  long long ld[COMFUSE_SPEC_MAX_PARAMS] = {0};
  for (int k = 0; k < an.n; ++k) {
    if (!an.live[k]) continue;
    const int op = an.nodes[k].op;
    if (op != COMFUSE_OP_ROWVEC && op != COMFUSE_OP_TENSOR) continue;
    const int q = an.nodes[k].param;
    if (!params || !params[q]) return COMFUSE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(params[q]) & 15u) return COMFUSE_ERR_ALIGNMENT;
    if (op == COMFUSE_OP_TENSOR) {
      ld[q] = (param_ld && param_ld[q] > 0) ? param_ld[q] : shape->N;
      if (ld[q] < shape->N) return COMFUSE_ERR_INVALID_ARG;
      if (ld[q] & 7) return COMFUSE_ERR_ALIGNMENT;
    }
  }
  for (size_t r = 0; r < an.row_outputs.size(); ++r)
    if (!row_out || !row_out[r]) return COMFUSE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(Y)) & 15u) return COMFUSE_ERR_ALIGNMENT;
  size_t need = 0;
  s = comfuse_gemm_spec_workspace_size(spec, shape, fused, &need);
  if (s != COMFUSE_OK) return s;
  if (need > 0 && (!workspace || workspace_bytes < need)) return COMFUSE_ERR_WORKSPACE;
  if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 15u)) return COMFUSE_ERR_ALIGNMENT;

  if (dc.fused && dc.match.kind == COMFUSE_EPI_BIAS_ACTIVATION) {
    const FusedMatch& m = dc.match;
    return run_gemm_elementwise(shape->batch, shape->M, shape->N, shape->K, shape->lda, shape->ldb, shape->ldy, shape->batch_stride_a,
                                shape->batch_stride_b, shape->batch_stride_y, A, B, Y, m.bias >= 0 ? params[m.bias] : nullptr, m.alpha,
                                m.activation, static_cast<cudaStream_t>(cuda_stream), (shape->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0);
  }
  if (dc.fused) {
    const FusedMatch& m = dc.match;
    const comfuse_gemm_desc_t d = fused_desc(*shape, m, m.residual >= 0 ? ld[m.residual] : shape->N);
    comfuse_epilogue_args_t a;
    std::memset(&a, 0, sizeof(a));
    auto prm = [&](int q) { return q >= 0 ? params[q] : nullptr; };
    a.bias = prm(m.bias); a.residual = prm(m.residual); a.gamma = prm(m.gamma); a.beta = prm(m.beta);
    if (m.kind == COMFUSE_EPI_BIAS_GELU_RES_RMSNORM_MAX) {
      char* scratch = static_cast<char*>(workspace) + dc.fused_inner_ws;
      const size_t rows = static_cast<size_t>(shape->batch) * shape->M;
      a.row_max = m.row_max_out >= 0 ? static_cast<float*>(row_out[m.row_max_out]) : reinterpret_cast<float*>(scratch);
      a.row_argmax = m.row_argmax_out >= 0 ? static_cast<int32_t*>(row_out[m.row_argmax_out]) : reinterpret_cast<int32_t*>(scratch + rows * 4);
    }
    return comfuse_gemm_epilogue(&d, A, B, Y, &a, workspace, dc.fused_inner_ws, cuda_stream);
  }

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (dc.on_chip) {
    // ONE fused kernel, the program's stages interpreted over the on-chip accumulator
    const StageBinding& bd = dc.stage_bind;
    const void* vecs[3] = {nullptr, nullptr, nullptr};
    for (int i = 0; i < bd.n_rowvec; ++i) vecs[i] = params[bd.rowvec_param[i]];
    StageProgram sp = dc.stage_prog;
    for (int r = 0; r < sp.n_row_out; ++r) sp.out[r].ptr = row_out[bd.row_out_pos[r]];
    const void* res = bd.tensor_param >= 0 ? params[bd.tensor_param] : nullptr;
    const long long ldres = bd.tensor_param >= 0 ? ld[bd.tensor_param] : shape->N;
    const bool b_nk = (shape->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0;
    if (try_generated) {
      // the best path: the kernel generated for this program; where it cannot be had (the compilation failed), the interpreter
      s = run_fused_program(shape->batch, shape->M, shape->N, shape->K, shape->lda, shape->ldb, shape->ldy, shape->batch_stride_a,
                            shape->batch_stride_b, shape->batch_stride_y, A, B, Y, sp, vecs, res, ldres, st, false, b_nk, true);
      if (s != COMFUSE_ERR_UNSUPPORTED || !dc.interp_ok) return s;
    }
    return run_fused_program(shape->batch, shape->M, shape->N, shape->K, shape->lda, shape->ldb, shape->ldy, shape->batch_stride_a,
                             shape->batch_stride_b, shape->batch_stride_y, A, B, Y, sp, vecs, res, ldres, st, false, b_nk, fused == 3);
  }

  // standard pathway: GEMM -> bf16 Z in the workspace -> row program
  RowProgram P;
  std::memset(&P, 0, sizeof(P));
  int ni, ns;
  s = lower_row_program(an, shape->N, P, ni, ns);
  if (s != COMFUSE_OK) return s;
  s = gemm_to_bf16(shape->batch, shape->M, shape->N, shape->K, shape->lda, shape->ldb, shape->batch_stride_a, shape->batch_stride_b, A, B,
                   workspace, st, (shape->flags & COMFUSE_FLAG_B_ROW_MAJOR_NK) != 0);
  if (s != COMFUSE_OK) return s;
  P.batch = shape->batch; P.M = shape->M; P.N = shape->N;
  P.Z = static_cast<const uint16_t*>(workspace);
  P.Y = static_cast<uint16_t*>(Y);
  P.ldy = shape->ldy;
  P.batch_stride_y = shape->batch > 1 ? shape->batch_stride_y : 0;
  for (int q = 0; q < spec->n_params; ++q) {
    P.params[q] = params ? static_cast<const uint16_t*>(params[q]) : nullptr;
    P.param_ld[q] = ld[q];
  }
  for (int r = 0; r < P.n_row_out; ++r) P.row_out[r] = row_out[r];
  return launch_row_program(P, st) == cudaSuccess ? COMFUSE_OK : COMFUSE_ERR_CUDA;
}

}  // extern "C"
