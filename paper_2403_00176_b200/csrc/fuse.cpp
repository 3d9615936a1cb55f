// RDP-enabled operator fusion (Section 4.2) and partition at execution-determined operators
// (Section 4.3).  A group is one anchor (GEMM / conv / attention) or none, followed by a chain of
// elementwise operators whose index space RDP proves equal to the anchor's output (dims equal as
// lattice values, or each broadcast dim resolved to "1" vs "same"), plus at most one trailing row
// reduction.  When a broadcast pair is unresolved the operator stays unfused and the number of
// versions that fusion would have needed (2^d) is recorded.
#include <algorithm>
#include <functional>
#include <set>

#include "engine.h"

namespace sod2 {

const char* gkind_name(GKind k) {
  switch (k) {
    case GKind::GEMM: return "gemm";
    case GKind::ATTENTION: return "attention";
    case GKind::LAYERNORM: return "layernorm";
    case GKind::CHAIN: return "chain";
    case GKind::TOPK_KEEP: return "topk_keep";
    case GKind::NONZERO: return "nonzero";
    case GKind::CONV: return "conv";
    case GKind::GAP: return "gap";
    case GKind::GATE: return "gate";
    case GKind::SWITCH: return "switch";
    case GKind::COMBINE: return "combine";
    case GKind::LAYOUT: return "layout";
    case GKind::BMM: return "bmm";
    case GKind::SUMSQ: return "sumsq";
    case GKind::TOPK: return "topk";
    case GKind::GATHER: return "gather";
    case GKind::FILL: return "fill";
    case GKind::RESIZE: return "resize";
    default: return "unsupported";
  }
}

namespace {

bool is_elementwise(const std::string& op) {
  return op == "Add" || op == "Sub" || op == "Mul" || op == "Div" || op == "Relu" || op == "Gelu" || op == "Sigmoid";
}
bool is_unary(const std::string& op) { return op == "Relu" || op == "Gelu" || op == "Sigmoid"; }
bool is_view_op(const std::string& op) { return op == "Reshape" || op == "Transpose" || op == "Slice"; }

struct Fuser {
  Compiled& c;
  Graph& g;
  std::vector<int> assigned;  // node -> group index (-1 none)
  explicit Fuser(Compiled& cc) : c(cc), g(cc.g), assigned(cc.g.nodes.size(), -1) {}

  bool same_shape(int t1, int t2) const {
    const ShapeVal &a = g.tensors[t1].S, &b = g.tensors[t2].S;
    if (a.rank < 0 || a.rank != b.rank) return false;
    for (int i = 0; i < a.rank; ++i) if (!a.dims[i].known() || a.dims[i] != b.dims[i]) return false;
    return true;
  }
  // t2 broadcasts into t1's index space with every dim pair resolved to "1" or "same"
  bool resolved_bcast(int t1, int t2) const {
    const ShapeVal &a = g.tensors[t1].S, &b = g.tensors[t2].S;
    if (a.rank < 0 || b.rank < 0 || b.rank > a.rank) return false;
    for (int i = 0; i < b.rank; ++i) {
      const Dim &da = a.dims[a.rank - b.rank + i], &db = b.dims[i];
      if (!da.known() || !db.known()) return false;
      bool one = db.e.is_const() && db.e.const_value() == 1;
      if (!one && da != db) return false;
    }
    return true;
  }
  // the real data consumers of a tensor (Shape readers only look at the S-map, which RDP folded)
  std::vector<int> data_consumers(int t) const {
    std::vector<int> r;
    for (int n : g.tensors[t].consumers) if (!c.node_folded[n] || is_view_op(g.nodes[n].op)) r.push_back(n);
    return r;
  }
  int sole_consumer(int t) const {
    if (g.tensors[t].is_output) return -1;
    std::vector<int> cs = data_consumers(t);
    if (cs.size() != 1 || assigned[cs[0]] >= 0 || c.node_folded[cs[0]]) return -1;
    return cs[0];
  }
  bool depends_on(int tensor, const std::set<int>& nodes) const {
    // is `tensor` a descendant of any node in `nodes`?
    std::vector<int> stack = {tensor};
    std::set<int> seen;
    while (!stack.empty()) {
      int t = stack.back(); stack.pop_back();
      int p = g.tensors[t].producer;
      if (p < 0 || seen.count(p)) continue;
      if (nodes.count(p)) return true;
      seen.insert(p);
      for (int i : g.nodes[p].ins) stack.push_back(i);
    }
    return false;
  }
  bool is_const_vec(int t, const Dim& n) const {
    const Tensor& T = g.tensors[t];
    return T.kind == TKind::CONST && T.S.rank == 1 && T.S.dims[0] == n;
  }

  void finish(Group& G) {
    std::set<int> inside(G.nodes.begin(), G.nodes.end());
    std::set<int> produced;
    for (int n : G.nodes) for (int o : g.nodes[n].outs) produced.insert(o);
    std::set<int> ins;
    for (int n : G.nodes)
      for (int i : g.nodes[n].ins)
        if (!produced.count(i) && g.tensors[i].kind != TKind::ICONST && g.tensors[i].kind != TKind::FCONST &&
            g.tensors[i].V.kind != ValueVal::KNOWN)
          ins.insert(i);
    G.ext_in.assign(ins.begin(), ins.end());
    for (int o : produced) {
      bool ext = g.tensors[o].is_output;
      for (int cn : g.tensors[o].consumers) if (!inside.count(cn)) ext = true;
      if (ext) G.ext_out.push_back(o);
    }
    int gi = static_cast<int>(c.groups.size());
    for (int n : G.nodes) { assigned[n] = gi; g.nodes[n].group = gi; }
    c.groups.push_back(G);
  }

  // epilogue absorption shared by GEMM and conv anchors
  void absorb_epilogue(Group& G, int cur, bool channel_bias) {
    const bool fuse = !(c.flags & OPT_NO_FUSION);
    std::set<int> inside(G.nodes.begin(), G.nodes.end());
    while (fuse) {
      int nx = sole_consumer(cur);
      if (nx < 0) break;
      const Node& n = g.nodes[nx];
      if (n.op == "Add") {
        int other = n.ins[0] == cur ? n.ins[1] : n.ins[0];
        const ShapeVal& cs = g.tensors[cur].S;
        bool bias_ok = !channel_bias && G.bias < 0 && G.act == 0 && G.res < 0 && cs.rank >= 1 && is_const_vec(other, cs.dims[cs.rank - 1]);
        if (bias_ok) { G.bias = other; }
        else if (G.res < 0 && G.act2 == 0 && same_shape(cur, other) && !depends_on(other, inside)) { G.res = other; }
        else break;
      } else if (n.op == "Gelu" || n.op == "Relu") {
        int code = n.op == "Gelu" ? 1 : 2;
        if (G.res < 0 && G.act == 0) G.act = code;
        else if (G.res >= 0 && G.act2 == 0) G.act2 = code;
        else break;
      } else if (n.op == "LayerNormalization" && G.kind == GKind::GEMM && g.tensors[cur].dtype == DType::F32 && n.attr_i("axis", -1) == -1) {
        const ShapeVal& cs = g.tensors[cur].S;
        const Dim& nd = cs.dims[cs.rank - 1];
        if (!(nd.e.is_const() && nd.e.const_value() <= 128 && nd.e.const_value() % 32 == 0)) break;
        G.has_ln = 1; G.gamma = n.ins[1]; G.beta = n.ins[2]; G.eps = static_cast<float>(n.attr_f("epsilon", 1e-5));
        G.nodes.push_back(nx); inside.insert(nx);
        cur = n.outs[0];
        break;
      } else if (n.op == "LayerNormalization" && G.kind == GKind::GEMM && g.tensors[cur].dtype == DType::BF16 && n.attr_i("axis", -1) == -1 &&
                 G.act2 == 0 && (c.flags & OPT_SPLITK_LN)) {
        // bf16 GEMM (+bias, +residual) -> LayerNorm: the GEMM runs split along K into an fp32 workspace and
        // the finishing kernel applies bias, residual and the normalisation (row width must fit a warp)
        const ShapeVal& cs = g.tensors[cur].S;
        const Dim& nd = cs.dims[cs.rank - 1];
        if (!(nd.e.is_const() && nd.e.const_value() <= 1024 && nd.e.const_value() % 8 == 0)) break;
        if (G.act != 0) break;
        if (g.tensors[n.ins[1]].kind != TKind::CONST || g.tensors[n.ins[2]].kind != TKind::CONST) break;
        G.has_ln = 1; G.gamma = n.ins[1]; G.beta = n.ins[2]; G.eps = static_cast<float>(n.attr_f("epsilon", 1e-5));
        G.nodes.push_back(nx); inside.insert(nx);
        cur = n.outs[0];
        break;
      } else break;
      G.nodes.push_back(nx);
      inside.insert(nx);
      cur = n.outs[0];
    }
    G.out = cur;
  }

  bool try_attention(int nid) {
    if (c.flags & OPT_NO_FUSION) return false;
    const Node& n = g.nodes[nid];
    if (g.tensors[n.ins[0]].kind == TKind::CONST || g.tensors[n.ins[1]].kind == TKind::CONST) return false;
    Group G;
    G.kind = GKind::ATTENTION;
    G.nodes = {nid};
    int cur = n.outs[0];
    int nx = sole_consumer(cur);
    if (nx >= 0 && g.nodes[nx].op == "Mul") {
      const Node& m = g.nodes[nx];
      int other = m.ins[0] == cur ? m.ins[1] : m.ins[0];
      if (g.tensors[other].kind != TKind::FCONST) return false;
      G.scale = static_cast<float>(g.tensors[other].fdata);
      G.nodes.push_back(nx);
      cur = m.outs[0];
      nx = sole_consumer(cur);
    }
    if (nx < 0 || g.nodes[nx].op != "Softmax" || g.nodes[nx].attr_i("axis", -1) != -1) return false;
    G.nodes.push_back(nx);
    cur = g.nodes[nx].outs[0];
    nx = sole_consumer(cur);
    if (nx < 0 || g.nodes[nx].op != "MatMul" || g.nodes[nx].ins[0] != cur) return false;
    if (g.tensors[g.nodes[nx].ins[1]].kind == TKind::CONST) return false;
    G.nodes.push_back(nx);
    G.q = n.ins[0]; G.k = n.ins[1]; G.v = g.nodes[nx].ins[1];
    G.out = g.nodes[nx].outs[0];
    finish(G);
    return true;
  }

  bool try_topk_keep(int nid) {
    // ReduceSumSquare(y) -> TopK(order=index) -> [Reshape idx] -> Gather(y, idx, axis=1)
    if (c.flags & OPT_NO_FUSION) return false;
    const Node& n = g.nodes[nid];
    if (n.attr_i("axis", -1) != -1 && n.attr_i("axis", -1) != g.tensors[n.ins[0]].S.rank - 1) return false;
    int y = n.ins[0], sc = n.outs[0];
    std::vector<int> cs = data_consumers(sc);
    if (cs.size() != 1 || g.nodes[cs[0]].op != "TopK" || g.tensors[sc].is_output) return false;
    const Node& tk = g.nodes[cs[0]];
    if (tk.attr_s("order", "value") != "index" || tk.attr_i("largest", 1) != 1) return false;
    if (tk.outs.size() < 2 || !data_consumers(tk.outs[0]).empty() || g.tensors[tk.outs[0]].is_output) return false;
    int idx = tk.outs[1];
    // find Gather(y, view-of-idx)
    int gather = -1;
    std::function<void(int)> walk = [&](int t) {
      for (int cn : data_consumers(t)) {
        const Node& m = g.nodes[cn];
        if (m.op == "Reshape" && m.ins[0] == t) walk(m.outs[0]);
        else if (m.op == "Gather" && m.ins[1] == t && m.ins[0] == y && m.attr_i("axis", 0) == g.tensors[y].S.rank - 2) gather = cn;
      }
    };
    walk(idx);
    if (gather < 0) return false;
    Group G;
    G.kind = GKind::TOPK_KEEP;
    G.nodes = {nid, cs[0], gather};
    G.a = y; G.out = g.nodes[gather].outs[0]; G.out2 = idx; G.k = tk.ins[1];
    finish(G);
    return true;
  }

  bool try_gate(int nid) {
    // GlobalAveragePool -> Reshape -> MatMul(C x 1 const) -> Add(const) -> Greater(fconst)
    if (c.flags & OPT_NO_FUSION) return false;
    const Node& n = g.nodes[nid];
    int cur = n.outs[0];
    std::vector<int> chain = {nid};
    auto next_is = [&](const char* op) -> int {
      if (g.tensors[cur].is_output) return -1;
      std::vector<int> cs = data_consumers(cur);
      if (cs.size() != 1 || g.nodes[cs[0]].op != op || assigned[cs[0]] >= 0) return -1;
      return cs[0];
    };
    int r = next_is("Reshape");
    if (r < 0) return false;
    cur = g.nodes[r].outs[0];
    int mm = next_is("MatMul");
    if (mm < 0 || g.tensors[g.nodes[mm].ins[1]].kind != TKind::CONST) return false;
    const ShapeVal& ws = g.tensors[g.nodes[mm].ins[1]].S;
    if (ws.rank != 2 || !(ws.dims[1].e.is_const() && ws.dims[1].e.const_value() == 1)) return false;
    cur = g.nodes[mm].outs[0];
    int ad = next_is("Add");
    if (ad < 0) return false;
    int bias = g.nodes[ad].ins[0] == cur ? g.nodes[ad].ins[1] : g.nodes[ad].ins[0];
    if (g.tensors[bias].kind != TKind::CONST) return false;
    cur = g.nodes[ad].outs[0];
    int z = cur;
    // z may be a graph output too; Greater must be its only data consumer
    std::vector<int> cs = data_consumers(cur);
    if (cs.size() != 1 || g.nodes[cs[0]].op != "Greater") return false;
    int gr = cs[0];
    int thr = g.nodes[gr].ins[1];
    if (g.tensors[thr].kind != TKind::FCONST || g.tensors[thr].fdata != 0.0) return false;
    Group G;
    G.kind = GKind::GATE;
    G.nodes = {nid, r, mm, ad, gr};
    G.a = n.ins[0]; G.w = g.nodes[mm].ins[1]; G.bias = bias; G.out = g.nodes[gr].outs[0]; G.out2 = z;
    c.node_folded[r] = 1;  // the Reshape of the pooled vector lives inside the group
    finish(G);
    return true;
  }

  void chain_group(int nid) {
    Group G;
    G.kind = GKind::CHAIN;
    const bool fuse = !(c.flags & OPT_NO_FUSION);
    int cur;
    auto code_of = [&](const Node& n, int curt, int* operand) -> int {
      *operand = -1;
      if (n.op == "Relu") return 6;
      if (n.op == "Gelu") return 7;
      if (n.op == "Sigmoid") return 8;
      bool first = n.ins[0] == curt;
      *operand = first ? n.ins[1] : n.ins[0];
      if (n.op == "Add") return 0;
      if (n.op == "Mul") return 3;
      if (n.op == "Sub") return first ? 1 : 2;
      return first ? 4 : 5;  // Div
    };
    const Node& n0 = g.nodes[nid];
    if (n0.op == "Softmax" || n0.op == "LayerNormalization") {
      G.a = n0.ins[0];
      G.red = n0.op == "Softmax" ? 1 : 2;
      if (G.red == 2) { G.gamma = n0.ins[1]; G.beta = n0.ins[2]; G.eps = static_cast<float>(n0.attr_f("epsilon", 1e-5)); }
      G.nodes = {nid};
      G.out = n0.outs[0];
      finish(G);
      return;
    }
    // first op: pick in0 as the operand with the full output index space (or the unary input)
    int out0 = n0.outs[0];
    int operand;
    if (is_unary(n0.op)) { G.a = n0.ins[0]; }
    else {
      // the larger-rank / non-constant operand leads
      int l = n0.ins[0], r = n0.ins[1];
      bool l_full = same_shape(l, out0), r_full = same_shape(r, out0);
      G.a = (l_full || !r_full) ? l : r;
    }
    G.chain_ops.push_back(code_of(n0, G.a, &operand));
    G.chain_operands.push_back(operand);
    G.nodes = {nid};
    int unres = static_cast<int>(n0.attr_i("unresolved_bcast", 0));
    int vbits = 0;                      // unresolved extent pairs fused across (multi-version fusion)
    cur = out0;
    while (fuse && G.chain_ops.size() < 8) {
      int nx = sole_consumer(cur);
      if (nx < 0) break;
      const Node& n = g.nodes[nx];
      if (is_elementwise(n.op)) {
        int opd;
        int code = code_of(n, cur, &opd);
        if (opd >= 0) {
          // RDP-enabled fusion: legal only if the operand provably shares the index space or
          // broadcasts into it dim by dim
          // RDP-enabled fusion: legal only if both the running value and the operand provably
          // share the output's index space or broadcast into it dim by dim ("1" or "same")
          if (!(resolved_bcast(n.outs[0], opd) && resolved_bcast(n.outs[0], cur))) {
            int u = static_cast<int>(n.attr_i("unresolved_bcast", 0));
            // Multi-version fusion (Section 4.2): d unresolved extent pairs need 2^d fused versions.  The
            // chain kernel is parametric in its strides, so a "version" is a stride table and is chosen at
            // bind time, when the extents are known (a broadcast extent reads with stride 0); the bind-time
            // assertions reject pairs that are neither equal nor 1.  Off by default: without the flag the
            // operators stay unfused, which is what RDP's resolution of the extents saves.
            const bool all_known = g.tensors[n.outs[0]].S.fully_known() && g.tensors[opd].S.fully_known() && g.tensors[cur].S.fully_known();
            if (u && (c.flags & OPT_MULTI_VERSION) && all_known && vbits + u <= 16) { vbits += u; }
            else {
              if (u) { G.versions = std::max(G.versions, 1 << u); }
              break;
            }
          }
          std::set<int> inside(G.nodes.begin(), G.nodes.end());
          if (depends_on(opd, inside)) break;
        }
        G.chain_ops.push_back(code);
        G.chain_operands.push_back(opd);
        G.nodes.push_back(nx);
        cur = n.outs[0];
      } else if ((n.op == "Softmax" || n.op == "LayerNormalization") && n.attr_i("axis", -1) == -1 && n.ins[0] == cur) {
        G.red = n.op == "Softmax" ? 1 : 2;
        if (G.red == 2) { G.gamma = n.ins[1]; G.beta = n.ins[2]; G.eps = static_cast<float>(n.attr_f("epsilon", 1e-5)); }
        G.nodes.push_back(nx);
        cur = n.outs[0];
        break;
      } else break;
    }
    if (unres + vbits) G.versions = std::max(G.versions, 1 << (unres + vbits));
    G.out = cur;
    finish(G);
  }

  // 3c. LayerNorm folded into the neighbouring GEMMs (RDP-enabled fusion, Section 4.2: the row width is a known
  // constant and the operands' index spaces are proven equal, so the normalisation distributes over the product):
  //   LayerNorm(x) W + b = rstd_i (x_i . (gamma o W)) - rstd_i mean_i (gamma^T W) + (beta^T W + b).
  // A bf16 LayerNorm whose input is the output of a GEMM group and whose every consumer is a GEMM group (as the A
  // operand or as the residual) is removed: the producing GEMM also writes per-row statistics, the consumers read
  // the raw rows and normalise in their epilogues; the normalised tensor becomes an alias of the raw one and is
  // never stored.  One kernel and one round trip of the tensor through memory less per LayerNorm.
  void fold_layernorms() {
    c.stats_width.assign(g.tensors.size(), 0);
    if (!(c.flags & OPT_LN_FOLD) || (c.flags & (OPT_NO_FUSION | OPT_SPLITK_LN))) return;
    std::vector<char> drop(c.groups.size(), 0);
    for (size_t li = 0; li < c.groups.size(); ++li) {
      const Group L = c.groups[li];
      if (L.kind != GKind::LAYERNORM) continue;
      const int raw = L.a, ln = L.out;
      const Tensor& R = g.tensors[raw];
      if (R.dtype != DType::BF16 || R.kind != TKind::VALUE || R.is_output || g.tensors[ln].is_output) continue;
      if (c.storage[raw].kind != Storage::ROOT || c.storage[ln].kind != Storage::ROOT) continue;
      if (R.S.rank < 1 || !R.S.dims[R.S.rank - 1].known() || !R.S.dims[R.S.rank - 1].e.is_const()) continue;
      const int64_t D = R.S.dims[R.S.rank - 1].e.const_value();
      if (D % 64 || D < 64 || D > 4096) continue;
      if (!is_const_vec(L.gamma, R.S.dims[R.S.rank - 1]) || !is_const_vec(L.beta, R.S.dims[R.S.rank - 1])) continue;
      if (g.tensors[L.gamma].dtype != DType::BF16 || g.tensors[L.beta].dtype != DType::BF16) continue;
      // the producer: a plain bf16 GEMM group (no activation: the statistics are taken of the stored rows)
      const int pn = R.producer;
      if (pn < 0 || assigned[pn] < 0) continue;
      const int pi = assigned[pn];
      const Group& P = c.groups[pi];
      if (P.kind != GKind::GEMM || P.out != raw || P.has_ln || P.act || P.act2 || P.ln_a >= 0 || g.tensors[P.a].dtype != DType::BF16) continue;
      // the consumers
      std::vector<std::pair<int, int>> uses;   // (group, 1 = A operand, 2 = residual)
      bool ok = true;
      for (int cn : data_consumers(ln)) {
        const int gi = assigned[cn];
        if (gi < 0) { ok = false; break; }
        const Group& G = c.groups[gi];
        if (G.kind != GKind::GEMM || G.has_ln || G.ln_a >= 0 || G.ln_res >= 0 || g.tensors[G.w].dtype != DType::BF16) { ok = false; break; }
        for (auto& u : uses) if (u.first == gi) ok = false;                       // one role per group
        if (!ok) break;
        if (cn == G.nodes[0] && G.a == ln && g.nodes[cn].ins[0] == ln && G.res != ln) {
          if (G.res >= 0 || G.emit_stats || G.act2) { ok = false; break; }
          uses.push_back({gi, 1});
        } else if (G.res == ln && G.a != ln && G.act == 0 && G.act2 == 0) {
          const ShapeVal& ws = g.tensors[G.w].S;
          if (!(ws.dims[1].e.is_const() && ws.dims[1].e.const_value() == D)) { ok = false; break; }
          uses.push_back({gi, 2});
        } else { ok = false; break; }
      }
      if (!ok || uses.empty()) continue;
      c.groups[pi].emit_stats = 1;
      c.stats_width[raw] = static_cast<int>(D);
      for (auto& u : uses) {
        Group& G = c.groups[u.first];
        (u.second == 1 ? G.ln_a : G.ln_res) = raw;
        G.ln_gamma = L.gamma; G.ln_beta = L.beta; G.ln_eps = L.eps;
        for (int t : {L.gamma, L.beta}) if (std::find(G.ext_in.begin(), G.ext_in.end(), t) == G.ext_in.end()) G.ext_in.push_back(t);
      }
      c.storage[ln] = Storage{Storage::ALIAS, L.nodes[0], raw, -1, 0};
      // the LayerNorm operator now runs inside its consumers; it is reported with the first of them, and the
      // dependency walk passes through it to the producer of the raw rows
      c.groups[uses[0].first].nodes.push_back(L.nodes[0]);
      assigned[L.nodes[0]] = -1;
      g.nodes[L.nodes[0]].group = uses[0].first;
      drop[li] = 1;
    }
    // remove the folded groups
    std::vector<int> remap(c.groups.size(), -1);
    std::vector<Group> kept;
    for (size_t gi = 0; gi < c.groups.size(); ++gi) if (!drop[gi]) { remap[gi] = static_cast<int>(kept.size()); kept.push_back(c.groups[gi]); }
    if (kept.size() == c.groups.size()) return;
    c.groups.swap(kept);
    for (auto& a : assigned) if (a >= 0) a = remap[a];
    for (auto& n : g.nodes) if (n.group >= 0) n.group = remap[n.group];
  }

  Status run() {
    // 1. nodes evaluated by RDP itself: every output has a fully known value map (shape arithmetic)
    c.node_folded.assign(g.nodes.size(), 0);
    for (size_t i = 0; i < g.nodes.size(); ++i) {
      bool all = !g.nodes[i].outs.empty();
      for (int o : g.nodes[i].outs) if (!g.tensors[o].V.all_known()) all = false;
      if (all) c.node_folded[i] = 1;
    }
    // 2. storage: view operators move no data
    c.storage.assign(g.tensors.size(), Storage());
    for (size_t i = 0; i < g.nodes.size(); ++i) {
      Node& n = g.nodes[i];
      if (c.node_folded[i]) { for (int o : n.outs) c.storage[o].kind = Storage::FOLDED; continue; }
      if (!is_view_op(n.op)) continue;
      c.node_folded[i] = 1;
      int in = n.ins[0], out = n.outs[0];
      const Tensor& I = g.tensors[in];
      int prod = I.producer;
      bool producer_computes = prod >= 0 && !is_view_op(g.nodes[prod].op);
      int n_data_cons = 0;
      for (int cn : I.consumers) if (!(g.nodes[cn].op == "Shape")) ++n_data_cons;
      if (n.op == "Transpose" && producer_computes && n_data_cons == 1 && !I.is_output && c.storage[in].kind == Storage::ROOT) {
        // the producer writes straight into the transposed layout
        c.storage[in].kind = Storage::VIEW_OF_OUTPUT;
        c.storage[in].node = static_cast<int>(i);
        c.storage[in].other = out;
      } else {
        c.storage[out].kind = Storage::VIEW_OF_INPUT;
        c.storage[out].node = static_cast<int>(i);
        c.storage[out].other = in;
      }
    }
    // 3. groups
    for (int nid : g.order) {
      if (assigned[nid] >= 0 || c.node_folded[nid]) continue;
      const Node& n = g.nodes[nid];
      const std::string& op = n.op;
      if (op == "MatMul") {
        const Tensor& B = g.tensors[n.ins[1]];
        if (B.kind == TKind::CONST && B.S.rank == 2) {
          Group G;
          G.kind = GKind::GEMM;
          G.nodes = {nid};
          G.a = n.ins[0]; G.w = n.ins[1];
          absorb_epilogue(G, n.outs[0], false);
          finish(G);
        } else if (!try_attention(nid)) {
          // MatMul of two activations outside the attention pattern (or in the unfused mode): stand-alone kernel
          Group G; G.kind = GKind::BMM; G.nodes = {nid}; G.a = n.ins[0]; G.w = n.ins[1]; G.out = n.outs[0];
          finish(G);
        }
      } else if (op == "Conv") {
        Group G;
        G.kind = GKind::CONV;
        G.nodes = {nid};
        G.a = n.ins[0]; G.w = n.ins[1]; G.bias = n.ins.size() > 2 ? n.ins[2] : -1;
        G.stride = static_cast<int>(n.attr_i("stride", 1)); G.pad = static_cast<int>(n.attr_i("pad", 0));
        G.ksize = static_cast<int>(g.tensors[n.ins[1]].S.dims[2].e.const_value());
        absorb_epilogue(G, n.outs[0], true);
        finish(G);
      } else if (is_elementwise(op) || op == "Softmax" || op == "LayerNormalization") {
        if (op == "LayerNormalization" && g.tensors[n.ins[0]].dtype == DType::BF16 && n.attr_i("axis", -1) == -1) {
          Group G;
          G.kind = GKind::LAYERNORM;
          G.nodes = {nid};
          G.a = n.ins[0]; G.gamma = n.ins[1]; G.beta = n.ins[2]; G.out = n.outs[0];
          G.eps = static_cast<float>(n.attr_f("epsilon", 1e-5));
          finish(G);
        } else chain_group(nid);
      } else if (op == "ReduceSumSquare") {
        if (!try_topk_keep(nid)) {
          Group G; G.nodes = {nid}; G.out = n.outs[0]; G.a = n.ins[0];
          const int rk = g.tensors[n.ins[0]].S.rank;
          if (n.attr_i("axis", -1) == -1 || n.attr_i("axis", -1) == rk - 1) G.kind = GKind::SUMSQ;
          else G.why = "ReduceSumSquare over an axis other than the last";
          finish(G);
        }
      } else if (op == "NonZero") {
        Group G; G.kind = GKind::NONZERO; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0]; finish(G);
      } else if (op == "GlobalAveragePool") {
        if (!try_gate(nid)) { Group G; G.kind = GKind::GAP; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0]; finish(G); }
      } else if (op == "ToChannelsLast" || op == "FromChannelsLast") {
        Group G; G.kind = GKind::LAYOUT; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0]; G.act = op == "FromChannelsLast";
        finish(G);
      } else if (op == "Switch") {
        Group G; G.kind = GKind::SWITCH; G.nodes = {nid}; G.a = n.ins[0]; G.gate = n.ins[1]; G.out = n.outs[0]; G.out2 = n.outs.size() > 1 ? n.outs[1] : -1;
        finish(G);
      } else if (op == "Combine") {
        Group G; G.kind = GKind::COMBINE; G.nodes = {nid}; G.a = n.ins[0]; G.res = n.ins[1]; G.gate = n.ins[2]; G.out = n.outs[0];
        finish(G);
      } else if (op == "Expand") {
        // a copy through the chain kernel: the operand is read with stride 0 along the dims it broadcasts over
        Group G; G.kind = GKind::CHAIN; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0];
        finish(G);
      } else if (op == "Resize" || op == "Upsample") {
        Group G; G.kind = GKind::RESIZE; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0];
        if (n.attr_s("mode", "nearest") != "nearest") { G.kind = GKind::UNSUPPORTED; G.why = "Resize: only nearest-neighbour interpolation has an executor"; }
        finish(G);
      } else if (op == "Range" || op == "ConstantOfShape") {
        Group G; G.kind = GKind::FILL; G.nodes = {nid}; G.out = n.outs[0]; G.act = op == "Range";
        G.scale = static_cast<float>(n.attr_f("value", 0.0));
        finish(G);
      } else if (op == "TopK" && n.outs.size() == 2) {
        Group G; G.nodes = {nid}; G.a = n.ins[0]; G.out = n.outs[0]; G.out2 = n.outs[1];
        const int rk = g.tensors[n.ins[0]].S.rank;
        if (n.attr_i("axis", -1) == -1 || n.attr_i("axis", -1) == rk - 1) {
          G.kind = GKind::TOPK;
          G.act = n.attr_s("order", "value") == "value";     // 1: by rank, 0: kept positions ascending
          G.act2 = static_cast<int>(n.attr_i("largest", 1));
        } else G.why = "TopK over an axis other than the last";
        finish(G);
      } else if (op == "Gather" && g.tensors[n.ins[1]].dtype == DType::I64) {
        Group G; G.kind = GKind::GATHER; G.nodes = {nid}; G.a = n.ins[0]; G.k = n.ins[1]; G.out = n.outs[0];
        G.stride = static_cast<int>(n.attr_i("axis", 0));
        finish(G);
      } else {
        Group G; G.nodes = {nid}; G.why = "no kernel for " + op; G.out = n.outs.empty() ? -1 : n.outs[0];
        finish(G);
      }
    }
    // 3b. index-indirect regrouping: where the executed branch of a Switch is consumed only by
    // convolutions (as input or residual), the skipped branch only by the matching Combine, and the
    // Combine's executed operand is a convolution output, nothing is copied at the Switch: the
    // convolutions read the Switch input through the executed-id list and the last one writes into the
    // Combine output at those ids; the Combine only moves the skipped samples.
    if (!(c.flags & (OPT_COPY_REGROUP | OPT_NO_FUSION))) {
      auto conv_ok = [&](const Group& G) {
        if (G.kind != GKind::CONV) return false;
        const Tensor& W = g.tensors[G.w];
        return W.dtype == DType::BF16 && W.S.rank == 4 && W.S.dims[0].e.is_const() && W.S.dims[1].e.is_const() &&
               W.S.dims[0].e.const_value() % 64 == 0 && W.S.dims[1].e.const_value() % 64 == 0;
      };
      for (size_t si = 0; si < c.groups.size(); ++si) {
        const Group& S = c.groups[si];
        if (S.kind != GKind::SWITCH || S.out2 < 0) continue;
        const int e = S.out, sk = S.out2, x = S.a;
        if (g.tensors[e].is_output || g.tensors[sk].is_output) continue;
        int cb = -1;
        for (size_t ci = 0; ci < c.groups.size(); ++ci)
          if (c.groups[ci].kind == GKind::COMBINE && c.groups[ci].gate == S.gate && c.groups[ci].res == sk) cb = static_cast<int>(ci);
        if (cb < 0) continue;
        const Group& C = c.groups[cb];
        bool ok = true;
        for (int cn : data_consumers(e)) {
          const int gi = assigned[cn];
          if (gi < 0 || !conv_ok(c.groups[gi])) { ok = false; break; }
          const Group& G = c.groups[gi];
          if (!((G.a == e && g.nodes[G.nodes[0]].ins[0] == e) || G.res == e)) { ok = false; break; }
          if (G.bias == e || G.w == e) { ok = false; break; }
        }
        std::vector<int> sc = data_consumers(sk);
        if (sc.size() != 1 || assigned[sc[0]] != cb) ok = false;
        const int ye = C.a;
        const int yp = g.tensors[ye].producer;
        if (yp < 0 || assigned[yp] < 0 || !conv_ok(c.groups[assigned[yp]]) || c.groups[assigned[yp]].out != ye) ok = false;
        std::vector<int> yc = data_consumers(ye);
        if (yc.size() != 1 || assigned[yc[0]] != cb || g.tensors[ye].is_output || g.tensors[C.out].is_output) ok = false;
        if (c.storage[e].kind != Storage::ROOT || c.storage[sk].kind != Storage::ROOT || c.storage[ye].kind != Storage::ROOT) ok = false;
        if (!ok) continue;
        c.storage[e] = Storage{Storage::INDIRECT_IN, S.nodes[0], x, S.gate, 0};
        c.storage[sk] = Storage{Storage::INDIRECT_IN, S.nodes[0], x, S.gate, 1};
        c.storage[ye] = Storage{Storage::INDIRECT_OUT, C.nodes[0], C.out, S.gate, 0};
        // In place: if nothing else reads the Switch input (besides the gate that decided the Switch and
        // the Switch itself), the Combine output takes over its storage; the skipped samples then never
        // move and the executed ones are overwritten by the block's last convolution, which reads its
        // residual tile before it stores the same tile.  Not with OPT_NO_REUSE, which promises that every
        // intermediate stays readable after the run.
        if (!(c.flags & OPT_NO_REUSE) && !g.tensors[x].is_output && g.tensors[x].kind == TKind::VALUE &&
            (c.storage[x].kind == Storage::ROOT || c.storage[x].kind == Storage::ALIAS)) {
          bool only = true;
          const int gate_prod = g.tensors[S.gate].producer;
          const int gate_group = gate_prod >= 0 ? assigned[gate_prod] : -1;
          for (int cn : data_consumers(x)) {
            const int gi = assigned[cn];
            if (gi == static_cast<int>(si)) continue;
            if (gi >= 0 && gi == gate_group && c.groups[gi].kind == GKind::GATE) continue;
            only = false;
          }
          // the block's first convolution must not be the one that writes in place (it reads halos of x)
          const Group& last = c.groups[assigned[yp]];
          if (last.a == e) only = false;
          if (only && c.storage[C.out].kind == Storage::ROOT) c.storage[C.out] = Storage{Storage::ALIAS, C.nodes[0], x, S.gate, 0};
        }
      }
    }
    fold_layernorms();
    // 4. partition at execution-determined operators (Section 4.3): a node's sub-graph index is
    // one more than that of any execution-determined producer it (transitively) depends on.
    std::vector<int> tsub(g.tensors.size(), 0);
    int maxsub = 0;
    for (int nid : g.order) {
      Node& n = g.nodes[nid];
      int s = 0;
      for (int i : n.ins) s = std::max(s, tsub[i]);
      n.subgraph = s;
      bool edo_count = n.op == "NonZero" || n.op == "Switch" || n.op == "Combine";
      for (int o : n.outs) tsub[o] = s + (edo_count ? 1 : 0);
      maxsub = std::max(maxsub, s);
    }
    c.n_subgraphs = maxsub + 1;
    // 5. execution order of groups: topological, ties by first node
    size_t G = c.groups.size();
    std::vector<std::set<int>> deps(G);
    for (size_t gi = 0; gi < G; ++gi) {
      c.groups[gi].subgraph = 0;
      for (int n : c.groups[gi].nodes) c.groups[gi].subgraph = std::max(c.groups[gi].subgraph, g.nodes[n].subgraph);
      for (int t : c.groups[gi].ext_in) {
        // walk through views / folded nodes back to the producing group
        std::vector<int> st = {t};
        while (!st.empty()) {
          int x = st.back(); st.pop_back();
          int p = g.tensors[x].producer;
          if (p < 0) continue;
          if (assigned[p] >= 0) { if (assigned[p] != static_cast<int>(gi)) deps[gi].insert(assigned[p]); }
          else for (int i : g.nodes[p].ins) st.push_back(i);
        }
      }
    }
    std::vector<int> orderg, done(G, 0);
    for (size_t it = 0; it < G; ++it) {
      int pick = -1;
      for (size_t gi = 0; gi < G && pick < 0; ++gi) {
        if (done[gi]) continue;
        bool ready = true;
        for (int d : deps[gi]) if (!done[d]) ready = false;
        if (ready) pick = static_cast<int>(gi);
      }
      if (pick < 0) { c.err = "cyclic group dependencies"; return E_INTERNAL; }
      done[pick] = 1;
      orderg.push_back(pick);
    }
    // 5b. static execution planning (Section 4.3): the order of least peak memory inside each sub-graph
    if (!(c.flags & OPT_NO_SEP)) {
      std::vector<std::vector<int>> dv(G);
      for (size_t gi = 0; gi < G; ++gi) dv[gi].assign(deps[gi].begin(), deps[gi].end());
      plan_execution_order(&c, dv, &orderg);
    }
    std::vector<Group> sorted;
    std::vector<int> remap(G);
    for (size_t i = 0; i < G; ++i) { remap[orderg[i]] = static_cast<int>(i); sorted.push_back(c.groups[orderg[i]]); }
    c.groups.swap(sorted);
    for (auto& n : g.nodes) if (n.group >= 0) n.group = remap[n.group];
    // 6. weights that the tcgen05 GEMM wants K-major
    for (auto& G2 : c.groups)
      if (G2.kind == GKind::GEMM && g.tensors[G2.w].dtype == DType::BF16) {
        const ShapeVal& s = g.tensors[G2.w].S;
        const size_t wbytes = static_cast<size_t>(s.dims[0].e.const_value() * s.dims[1].e.const_value() * 2);
        bool found = false;
        for (size_t i = 0; i < c.packed_consts.size(); ++i)
          if (c.packed_consts[i] == G2.w) {
            const Compiled::PackedLn& e = c.packed_ln[i];
            if (G2.ln_a >= 0 ? (e.gamma == G2.ln_gamma && e.beta == G2.ln_beta && e.bias == G2.bias) : e.gamma < 0) found = true;
          }
        if (found) continue;
        c.packed_consts.push_back(G2.w);
        c.packed_off.push_back(c.packed_bytes);
        Compiled::PackedLn e;
        size_t bytes = (wbytes + 255) & ~size_t(255);
        if (G2.ln_a >= 0) {   // gamma-scaled copy followed by the two fp32 epilogue vectors
          e.gamma = G2.ln_gamma; e.beta = G2.ln_beta; e.bias = G2.bias;
          bytes += (static_cast<size_t>(s.dims[1].e.const_value()) * 8 + 255) & ~size_t(255);
        }
        c.packed_ln.push_back(e);
        c.packed_bytes += bytes;
      }
    // ... and convolution weights as [Cout, (dy, dx, ci)] for the implicit GEMM
    for (auto& G2 : c.groups)
      if (G2.kind == GKind::CONV && g.tensors[G2.w].dtype == DType::BF16) {
        if (std::find(c.packed_consts.begin(), c.packed_consts.end(), G2.w) == c.packed_consts.end()) {
          c.packed_consts.push_back(G2.w);
          c.packed_off.push_back(c.packed_bytes);
          c.packed_ln.push_back(Compiled::PackedLn());
          const auto& wd = g.tensors[G2.w].S.dims;
          size_t kk = static_cast<size_t>(wd[1].e.const_value() * wd[2].e.const_value() * wd[3].e.const_value());
          kk = (kk + 63) / 64 * 64;   // thin-channel convolutions pad K to a whole k-chunk
          const size_t bytes = static_cast<size_t>(wd[0].e.const_value()) * kk * 2;
          c.packed_bytes += (bytes + 255) & ~size_t(255);
        }
      }
    return OK;
  }
};

}  // namespace

// Table of the distinct extent expressions of the graph (canonical form as the key).
static void index_dim_exprs(Compiled* c) {
  const Graph& g = c->g;
  c->dim_exprs.clear();
  c->dim_expr_id.assign(g.tensors.size(), {});
  std::map<std::string, int> seen;
  for (size_t t = 0; t < g.tensors.size(); ++t) {
    const ShapeVal& s = g.tensors[t].S;
    if (s.rank < 0) continue;
    c->dim_expr_id[t].assign(s.rank, -1);
    for (int i = 0; i < s.rank; ++i) {
      if (!s.dims[i].known()) continue;
      const std::string key = e_str(g.cx, s.dims[i].e);
      auto it = seen.find(key);
      if (it == seen.end()) { it = seen.emplace(key, static_cast<int>(c->dim_exprs.size())).first; c->dim_exprs.push_back(s.dims[i].e); }
      c->dim_expr_id[t][i] = it->second;
    }
  }
}

// Parameters of the view operators, per tensor stored as a view.
static void index_view_params(Compiled* c) {
  const Graph& g = c->g;
  c->view_param.assign(g.tensors.size(), {});
  for (size_t t = 0; t < g.tensors.size() && t < c->storage.size(); ++t) {
    const Storage& st = c->storage[t];
    if ((st.kind != Storage::VIEW_OF_INPUT && st.kind != Storage::VIEW_OF_OUTPUT) || st.node < 0) continue;
    const Node& n = g.nodes[st.node];
    Compiled::ViewParam& vp = c->view_param[t];
    vp.op = n.op == "Transpose" ? 0 : n.op == "Reshape" ? 1 : 2;
    if (vp.op == 0) vp.a = n.attr_list("perm");
    if (vp.op == 2 && st.kind == Storage::VIEW_OF_INPUT && st.other >= 0) {
      const int rank = g.tensors[st.other].S.rank;
      for (int ax = 0; ax < rank; ++ax) {
        vp.a.push_back(n.attr_i("_start" + std::to_string(ax), 0));
        vp.b.push_back(n.attr_i("_step" + std::to_string(ax), 1));
      }
    }
  }
}

// Shape classes of the tensors (engine.h): keys are built from what binding and planning read.
static void index_shape_classes(Compiled* c) {
  const Graph& g = c->g;
  const size_t T = g.tensors.size();
  c->dim_class.assign(T, -1);
  c->view_class.assign(T, -1);
  std::map<std::vector<int>, int> dseen;
  for (size_t t = 0; t < T; ++t) {
    if (g.tensors[t].S.rank < 0) continue;
    auto it = dseen.emplace(c->dim_expr_id[t], static_cast<int>(dseen.size())).first;
    c->dim_class[t] = it->second;
  }
  c->n_dim_classes = static_cast<int>(dseen.size());
  std::map<std::vector<int64_t>, int> vseen;
  std::vector<char> state(T, 0);   // 1: being visited (a cycle cannot happen; guards against one all the same)
  std::function<int(int)> cls = [&](int t) -> int {
    if (c->view_class[t] >= 0 || state[t]) return c->view_class[t];
    if (t >= static_cast<int>(c->storage.size()) || c->dim_class[t] < 0) return -1;
    state[t] = 1;
    const Storage& st = c->storage[t];
    const Tensor& X = g.tensors[t];
    std::vector<int64_t> key{static_cast<int64_t>(st.kind), c->dim_class[t]};
    if (st.kind == Storage::FOLDED) { state[t] = 0; return -1; }
    if (st.kind == Storage::ROOT) {
      const bool channels_last = g.has_conv && X.S.rank == 4 && X.kind == TKind::VALUE && !X.is_output && (X.dtype == DType::BF16 || X.dtype == DType::F32);
      key.push_back(dtype_size(X.dtype));
      key.push_back(X.kind == TKind::CONST);
      key.push_back(channels_last);
      key.push_back(t < c->stats_width.size() ? c->stats_width[t] : 0);
    } else {
      const int oc = st.other >= 0 ? cls(st.other) : -1;
      if (oc < 0) { state[t] = 0; return -1; }
      key.push_back(oc);
      key.push_back(st.gate);
      key.push_back(st.list);
      const Compiled::ViewParam& vp = c->view_param[t];
      key.push_back(vp.op);
      key.push_back(static_cast<int64_t>(vp.a.size()));
      key.insert(key.end(), vp.a.begin(), vp.a.end());
      key.insert(key.end(), vp.b.begin(), vp.b.end());
    }
    auto it = vseen.emplace(key, static_cast<int>(vseen.size())).first;
    c->view_class[t] = it->second;
    state[t] = 0;
    return it->second;
  };
  for (size_t t = 0; t < T; ++t) cls(static_cast<int>(t));
  c->n_view_classes = static_cast<int>(vseen.size());
}

Status form_groups(Compiled* c) {
  Fuser f(*c);
  Status s = f.run();
  if (s == OK) { index_dim_exprs(c); index_view_params(c); index_shape_classes(c); }
  return s;
}

}  // namespace sod2
