// Graph text reader, operator classification (Table 2) and Rank-and-Dimension Propagation
// (Section 4.1, Algorithm 1) with the forward / backward Update functions and the Merge function.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <set>
#include <sstream>

#include "graph.h"

namespace sod2 {

// ------------------------------------------------------------------------------------ lattice
Dim meet(const Dim& a, const Dim& b) {
  if (a.kind == Dim::UNDEF) return b;
  if (b.kind == Dim::UNDEF) return a;
  if (a.kind == Dim::NAC || b.kind == Dim::NAC) return Dim::nac();
  return a.e == b.e ? a : Dim::nac();
}

const char* dyn_class_name(DynClass c) {
  switch (c) {
    case DynClass::ISDO: return "ISDO";
    case DynClass::ISDOS: return "ISDOS";
    case DynClass::ISVDOS: return "ISVDOS";
    default: return "EDO";
  }
}

bool classify_op(const std::string& op, DynClass* out) {
  static const std::map<std::string, DynClass> table = {
      // Input Shape Determined Output
      {"Shape", DynClass::ISDO}, {"ConstantOfShape", DynClass::ISDO}, {"EyeLike", DynClass::ISDO},
      // Input Shape Determined Output Shape (Table 2 row 2, "elementwise w/ broadcast" and "Reduce" expanded)
      {"Add", DynClass::ISDOS}, {"Sub", DynClass::ISDOS}, {"Mul", DynClass::ISDOS}, {"Div", DynClass::ISDOS},
      {"Greater", DynClass::ISDOS}, {"AveragePool", DynClass::ISDOS}, {"MaxPool", DynClass::ISDOS},
      {"GlobalAveragePool", DynClass::ISDOS}, {"Cast", DynClass::ISDOS}, {"Concat", DynClass::ISDOS},
      {"Conv", DynClass::ISDOS}, {"Gather", DynClass::ISDOS}, {"MatMul", DynClass::ISDOS},
      {"ReduceSumSquare", DynClass::ISDOS}, {"ReduceMean", DynClass::ISDOS}, {"ReduceSum", DynClass::ISDOS},
      {"Relu", DynClass::ISDOS}, {"Round", DynClass::ISDOS}, {"Sigmoid", DynClass::ISDOS}, {"Softmax", DynClass::ISDOS},
      // same class by the definitions of Section 3 (output shape is a function of input shapes only)
      {"Gelu", DynClass::ISDOS}, {"LayerNormalization", DynClass::ISDOS}, {"Transpose", DynClass::ISDOS},
      // internal storage-layout operators (inserted by the library, never written in a graph text)
      {"ToChannelsLast", DynClass::ISDOS}, {"FromChannelsLast", DynClass::ISDOS},
      // Input Shape & Value Determined Output Shape
      {"Expand", DynClass::ISVDOS}, {"GroupNormalization", DynClass::ISVDOS}, {"MaxUnpool", DynClass::ISVDOS},
      {"OneHot", DynClass::ISVDOS}, {"Range", DynClass::ISVDOS}, {"Reshape", DynClass::ISVDOS},
      {"Resize", DynClass::ISVDOS}, {"Slice", DynClass::ISVDOS}, {"TopK", DynClass::ISVDOS}, {"Upsample", DynClass::ISVDOS},
      // Execution Determined Output
      {"If", DynClass::EDO}, {"Loop", DynClass::EDO}, {"NonMaxSuppression", DynClass::EDO}, {"NonZero", DynClass::EDO},
      {"Switch", DynClass::EDO}, {"Combine", DynClass::EDO}};
  auto it = table.find(op);
  if (it == table.end()) return false;
  *out = it->second;
  return true;
}

int64_t Node::attr_i(const std::string& k, int64_t d) const {
  auto it = attrs.find(k);
  return it == attrs.end() ? d : std::strtoll(it->second.c_str(), nullptr, 10);
}
double Node::attr_f(const std::string& k, double d) const {
  auto it = attrs.find(k);
  return it == attrs.end() ? d : std::strtod(it->second.c_str(), nullptr);
}
std::string Node::attr_s(const std::string& k, const std::string& d) const {
  auto it = attrs.find(k);
  return it == attrs.end() ? d : it->second;
}
std::vector<int64_t> Node::attr_list(const std::string& k) const {
  std::vector<int64_t> r;
  auto it = attrs.find(k);
  if (it == attrs.end()) return r;
  std::stringstream ss(it->second);
  std::string tok;
  while (std::getline(ss, tok, ',')) r.push_back(std::strtoll(tok.c_str(), nullptr, 10));
  return r;
}

std::string shape_str(const Graph& g, const ShapeVal& s) {
  if (s.rank == RANK_UNDEF) return "undef";
  if (s.rank == RANK_NAC) return "nac";
  std::string r = "[";
  for (size_t i = 0; i < s.dims.size(); ++i) {
    if (i) r += ",";
    const Dim& d = s.dims[i];
    r += d.kind == Dim::UNDEF ? "undef" : d.kind == Dim::NAC ? "nac" : e_str(g.cx, d.e);
  }
  return r + "]";
}

// ------------------------------------------------------------------------------------ reader
static bool parse_dtype(const std::string& s, DType* t) {
  if (s == "f32") *t = DType::F32;
  else if (s == "bf16") *t = DType::BF16;
  else if (s == "i64") *t = DType::I64;
  else if (s == "bool") *t = DType::BOOL;
  else return false;
  return true;
}

static std::vector<std::string> split_ws(const std::string& s) {
  std::vector<std::string> r;
  std::istringstream is(s);
  std::string t;
  while (is >> t) r.push_back(t);
  return r;
}

static bool is_int(const std::string& s) {
  if (s.empty()) return false;
  size_t i = (s[0] == '-') ? 1 : 0;
  if (i == s.size()) return false;
  for (; i < s.size(); ++i) if (s[i] < '0' || s[i] > '9') return false;
  return true;
}

static int new_tensor(Graph* g, const std::string& name) {
  int id = static_cast<int>(g->tensors.size());
  g->tensors.emplace_back();
  g->tensors.back().name = name;
  g->tindex[name] = id;
  return id;
}

// "[a,b,c]" -> dims; '?' = undef; names must be declared symbols
static bool parse_dims(Graph* g, const std::string& txt, ShapeVal* s, std::string* err) {
  size_t l = txt.find('['), r = txt.rfind(']');
  if (l == std::string::npos || r == std::string::npos || r < l) { *err = "expected [dims]"; return false; }
  std::string body = txt.substr(l + 1, r - l - 1);
  s->dims.clear();
  std::stringstream ss(body);
  std::string tok;
  while (std::getline(ss, tok, ',')) {
    size_t a = tok.find_first_not_of(" \t"), b = tok.find_last_not_of(" \t");
    if (a == std::string::npos) continue;
    tok = tok.substr(a, b - a + 1);
    if (tok == "?") s->dims.push_back(Dim());
    else if (is_int(tok)) s->dims.push_back(Dim::c(std::strtoll(tok.c_str(), nullptr, 10)));
    else {
      int id = g->cx.find_symbol(tok);
      if (id < 0) { *err = "undeclared symbol '" + tok + "'"; return false; }
      s->dims.push_back(Dim::val(Expr::atom(id)));
    }
  }
  s->rank = static_cast<int>(s->dims.size());
  return true;
}

void insert_layout_nodes(Graph* g);

Status parse_ir(const char* text, size_t len, Graph* g) {
  std::string all(text, len);
  std::istringstream is(all);
  std::string line;
  int lineno = 0;
  auto fail = [&](const std::string& m) {
    g->err = "line " + std::to_string(lineno) + ": " + m;
    return E_PARSE;
  };
  while (std::getline(is, line)) {
    ++lineno;
    size_t h = line.find('#');
    if (h != std::string::npos) line = line.substr(0, h);
    std::string attrs_txt;
    size_t lb = line.find('{');
    if (lb != std::string::npos) {
      size_t rb = line.find('}', lb);
      if (rb == std::string::npos) return fail("unterminated attribute list");
      attrs_txt = line.substr(lb + 1, rb - lb - 1);
      line = line.substr(0, lb);
    }
    std::vector<std::string> tk = split_ws(line);
    if (tk.empty()) continue;
    const std::string& kw = tk[0];
    if (kw == "sym") {
      if (tk.size() != 2 && tk.size() != 4) return fail("sym NAME [min max]");
      int64_t lo = 1, hi = INT64_MAX;
      if (tk.size() == 4) {
        if (!is_int(tk[2]) || !is_int(tk[3])) return fail("bad symbol range");
        lo = std::strtoll(tk[2].c_str(), nullptr, 10);
        hi = std::strtoll(tk[3].c_str(), nullptr, 10);
      }
      if (g->cx.find_symbol(tk[1]) >= 0) return fail("symbol redeclared");
      g->user_syms.push_back(g->cx.symbol(tk[1], lo, hi, false));
    } else if (kw == "input" || kw == "const") {
      if (tk.size() < 4) return fail(kw + " NAME DTYPE [dims]");
      if (g->tensor(tk[1]) >= 0) return fail("tensor redeclared: " + tk[1]);
      DType dt;
      if (!parse_dtype(tk[2], &dt)) return fail("bad dtype " + tk[2]);
      std::string rest;
      for (size_t i = 3; i < tk.size(); ++i) rest += tk[i];
      int id = new_tensor(g, tk[1]);
      Tensor& t = g->tensors[id];
      t.dtype = dt;
      t.kind = kw == "input" ? TKind::INPUT : TKind::CONST;
      std::string err;
      if (rest == "?") { /* rank undefined */ }
      else if (!parse_dims(g, rest, &t.S, &err)) return fail(err);
      if (kw == "input") {
        t.io_index = static_cast<int>(g->inputs.size());
        g->inputs.push_back(id);
        t.V.kind = ValueVal::NAC;  // the value of a model input is not a constant of the analysis
      }
      else {
        if (!t.S.fully_known()) return fail("const needs a fully known shape");
        for (auto& d : t.S.dims) if (!d.e.is_const()) return fail("const needs integer dims");
        g->consts.push_back(id);
      }
    } else if (kw == "iconst" || kw == "fconst") {
      // iconst NAME i64 [n] = v...
      size_t eq = 0;
      while (eq < tk.size() && tk[eq] != "=") ++eq;
      if (eq == tk.size() || eq < 4) return fail(kw + " NAME DTYPE [dims] = values");
      if (g->tensor(tk[1]) >= 0) return fail("tensor redeclared: " + tk[1]);
      int id = new_tensor(g, tk[1]);
      Tensor& t = g->tensors[id];
      std::string rest;
      for (size_t i = 3; i < eq; ++i) rest += tk[i];
      std::string err;
      if (!parse_dims(g, rest, &t.S, &err)) return fail(err);
      int64_t numel = 1;
      for (auto& d : t.S.dims) { if (!d.known() || !d.e.is_const()) return fail("inline constant needs integer dims"); numel *= d.e.const_value(); }
      if (static_cast<int64_t>(tk.size() - eq - 1) != numel) return fail("value count does not match shape");
      if (kw == "iconst") {
        t.dtype = DType::I64;
        t.kind = TKind::ICONST;
        if (numel > 16) return fail("inline integer constant too large");
        t.V.kind = ValueVal::KNOWN;
        for (size_t i = eq + 1; i < tk.size(); ++i) {
          if (!is_int(tk[i])) return fail("bad integer " + tk[i]);
          int64_t v = std::strtoll(tk[i].c_str(), nullptr, 10);
          t.idata.push_back(v);
          t.V.elems.push_back(Dim::c(v));
        }
      } else {
        t.dtype = DType::F32;
        t.kind = TKind::FCONST;
        if (numel != 1) return fail("fconst must be a scalar");
        t.fdata = std::strtod(tk[eq + 1].c_str(), nullptr);
      }
    } else if (kw == "node") {
      size_t arrow = 0;
      while (arrow < tk.size() && tk[arrow] != "->") ++arrow;
      if (arrow == tk.size() || arrow < 2 || arrow + 1 >= tk.size()) return fail("node OP ins -> outs");
      Node n;
      n.op = tk[1];
      if (!classify_op(n.op, &n.cls)) { g->err = "line " + std::to_string(lineno) + ": unsupported operator " + n.op; return E_UNSUPPORTED_OP; }
      n.eff_cls = n.cls;
      int nid = static_cast<int>(g->nodes.size());
      for (size_t i = 2; i < arrow; ++i) {
        int t = g->tensor(tk[i]);
        if (t < 0) return fail("unknown tensor " + tk[i]);
        n.ins.push_back(t);
        g->tensors[t].consumers.push_back(nid);
      }
      for (size_t i = arrow + 1; i < tk.size(); ++i) {
        if (g->tensor(tk[i]) >= 0) return fail("tensor redefined: " + tk[i]);
        int t = new_tensor(g, tk[i]);
        g->tensors[t].producer = nid;
        g->tensors[t].out_slot = static_cast<int>(i - arrow - 1);
        n.outs.push_back(t);
      }
      for (auto& kv : split_ws(attrs_txt)) {
        size_t e = kv.find('=');
        if (e == std::string::npos) return fail("bad attribute " + kv);
        n.attrs[kv.substr(0, e)] = kv.substr(e + 1);
      }
      g->nodes.push_back(std::move(n));
    } else if (kw == "output") {
      if (tk.size() != 2) return fail("output NAME");
      int t = g->tensor(tk[1]);
      if (t < 0) return fail("unknown tensor " + tk[1]);
      g->tensors[t].is_output = true;
      g->tensors[t].io_index = static_cast<int>(g->outputs.size());
      g->outputs.push_back(t);
    } else {
      return fail("unknown statement '" + kw + "'");
    }
  }
  if (g->outputs.empty()) { g->err = "graph has no output"; return E_PARSE; }
  insert_layout_nodes(g);
  return OK;
}

// Layout selection for convolution graphs: the convolution groups work on channels-last storage
// (one pixel = one 128-byte row of 64 channels, which is what the tensor-core operand layout wants),
// while the ABI's inputs and outputs are NCHW.  Internal layout operators are inserted at rank-4
// float graph inputs consumed by a Conv and at rank-4 float graph outputs; they change storage
// only, every logical shape stays NCHW.
void insert_layout_nodes(Graph* g) {
  bool has_conv = false;
  for (auto& n : g->nodes) if (n.op == "Conv") has_conv = true;
  g->has_conv = has_conv;
  if (!has_conv) return;
  auto add_node = [&](const std::string& op, int in, int out) {
    Node n;
    n.op = op;
    classify_op(op, &n.cls);
    n.eff_cls = n.cls;
    n.ins = {in};
    n.outs = {out};
    int nid = static_cast<int>(g->nodes.size());
    g->tensors[in].consumers.push_back(nid);
    g->tensors[out].producer = nid;
    g->nodes.push_back(n);
    return nid;
  };
  // inputs: every non-Shape consumer reads the channels-last copy
  for (int t : std::vector<int>(g->inputs)) {
    Tensor& T = g->tensors[t];
    if (T.S.rank != 4 || (T.dtype != DType::BF16 && T.dtype != DType::F32)) continue;
    bool feeds_conv = false;
    for (int c : T.consumers) if (g->nodes[c].op == "Conv" && g->nodes[c].ins[0] == t) feeds_conv = true;
    if (!feeds_conv) continue;
    // a thin-channel image (e.g. RGB) stays NCHW: its convolution gathers patches itself (im2col)
    if (!T.S.dims[1].known() || !T.S.dims[1].e.is_const() || T.S.dims[1].e.const_value() % 64) continue;
    int cl = new_tensor(g, T.name + "@cl");
    g->tensors[cl].dtype = g->tensors[t].dtype;
    std::vector<int> cons = g->tensors[t].consumers;
    g->tensors[t].consumers.clear();
    for (int c : cons) {
      if (g->nodes[c].op == "Shape") { g->tensors[t].consumers.push_back(c); continue; }
      for (int& i : g->nodes[c].ins) if (i == t) i = cl;
      g->tensors[cl].consumers.push_back(c);
    }
    add_node("ToChannelsLast", t, cl);
  }
  // outputs: the producer writes an internal channels-last tensor, a layout operator fills the output
  for (int t : std::vector<int>(g->outputs)) {
    Tensor& T = g->tensors[t];
    if (T.producer < 0 || T.kind != TKind::VALUE) continue;
    const std::string& pop = g->nodes[T.producer].op;
    if (pop != "Conv" && pop != "Add" && pop != "Relu" && pop != "Combine" && pop != "Resize" && pop != "Upsample") continue;   // rank known only after RDP: restrict to conv-chain producers
    int cl = new_tensor(g, g->tensors[t].name + "@cl");
    Tensor& O = g->tensors[t];
    Tensor& C = g->tensors[cl];
    C.dtype = O.dtype;
    // the internal tensor takes over the producer and the consumers; the output keeps its name
    C.producer = O.producer;
    C.out_slot = O.out_slot;
    for (int& o : g->nodes[C.producer].outs) if (o == t) o = cl;
    C.consumers = O.consumers;
    for (int c : C.consumers) for (int& i : g->nodes[c].ins) if (i == t) i = cl;
    O.consumers.clear();
    O.producer = -1;
    add_node("FromChannelsLast", cl, t);
  }
}


// ------------------------------------------------------------------------------------ transfer helpers
namespace {

struct Rdp {
  Graph& g;
  Status st = OK;
  explicit Rdp(Graph& gg) : g(gg) {}

  void add_assert(const Expr& a, const Expr& b, const std::string& what) {
    if (a == b) return;
    for (auto& x : g.asserts) if (x.kind == 0 && ((x.a == a && x.b == b) || (x.a == b && x.b == a))) return;
    g.asserts.push_back({a, b, what, 0});
  }
  // An extent pair that RDP can resolve neither to "same" nor to "1" is legal only if the bound values do
  // (Section 4.2: the fused version is chosen once the extents are known).
  void add_bcast_assert(const Expr& a, const Expr& b, const std::string& what) {
    for (auto& x : g.asserts) if (x.kind == 1 && ((x.a == a && x.b == b) || (x.a == b && x.b == a))) return;
    g.asserts.push_back({a, b, what, 1});
  }

  // Move one component down the lattice. Two different constants from two inference sources must
  // be equal at run time (Section 4.1: producer- and consumer-side results "should be the same"):
  // keep the current one and record a bind-time assertion.
  bool refine(Dim& cur, const Dim& nw, const std::string& what) {
    if (nw.kind == Dim::UNDEF) return false;
    if (cur.kind == Dim::UNDEF) { cur = nw; return true; }
    if (cur == nw || cur.kind == Dim::NAC) return false;
    if (nw.kind == Dim::NAC) return false;
    if (cur.e.is_const() && nw.e.is_const()) { fail(E_SHAPE_CONFLICT, what + ": " + e_str(g.cx, cur.e) + " vs " + e_str(g.cx, nw.e)); return false; }
    add_assert(cur.e, nw.e, what);
    return false;
  }
  bool refine_shape(int t, const ShapeVal& nw) {
    Tensor& T = g.tensors[t];
    if (nw.rank == RANK_UNDEF) return false;
    bool ch = false;
    if (T.S.rank == RANK_UNDEF) { T.S.rank = nw.rank; T.S.dims.assign(nw.rank < 0 ? 0 : nw.rank, Dim()); ch = true; }
    if (T.S.rank != nw.rank) {
      if (T.S.rank >= 0 && nw.rank >= 0) fail(E_RANK_MISMATCH, "rank of " + T.name);
      return ch;
    }
    for (int i = 0; i < T.S.rank; ++i) ch |= refine(T.S.dims[i], nw.dims[i], "dim " + std::to_string(i) + " of " + T.name);
    return ch;
  }
  bool refine_value(int t, const ValueVal& nw) {
    Tensor& T = g.tensors[t];
    if (nw.kind == ValueVal::UNDEF) return false;
    if (T.V.kind == ValueVal::UNDEF) { T.V = nw; return true; }
    if (T.V.kind == ValueVal::NAC || nw.kind == ValueVal::NAC) return false;
    bool ch = false;
    if (T.V.elems.size() != nw.elems.size()) return false;
    for (size_t i = 0; i < nw.elems.size(); ++i) ch |= refine(T.V.elems[i], nw.elems[i], "value of " + T.name);
    return ch;
  }
  void fail(Status s, const std::string& m) {
    if (st == OK) { st = s; g.err = m; }
  }
  const ShapeVal& S(int t) const { return g.tensors[t].S; }
  const ValueVal& V(int t) const { return g.tensors[t].V; }

  static int norm_axis(int64_t ax, int rank) { return static_cast<int>(ax < 0 ? ax + rank : ax); }

  // ---- broadcast of two shapes (right aligned). unresolved = number of dim pairs RDP cannot
  // resolve to "1" or "same" (each doubles the number of code versions, Section 4.2).
  ShapeVal bcast(const ShapeVal& a, const ShapeVal& b, const std::string& who, int* unresolved) {
    ShapeVal o;
    if (a.rank == RANK_NAC || b.rank == RANK_NAC) { o.rank = RANK_NAC; return o; }
    if (a.rank < 0 || b.rank < 0) return o;
    o.rank = std::max(a.rank, b.rank);
    o.dims.resize(o.rank);
    for (int i = 0; i < o.rank; ++i) {
      int ia = i - (o.rank - a.rank), ib = i - (o.rank - b.rank);
      Dim da = ia >= 0 ? a.dims[ia] : Dim::c(1), db = ib >= 0 ? b.dims[ib] : Dim::c(1);
      auto is1 = [](const Dim& d) { return d.known() && d.e.is_const() && d.e.const_value() == 1; };
      if (da.kind == Dim::NAC || db.kind == Dim::NAC) {
        o.dims[i] = is1(da) ? db : is1(db) ? da : Dim::nac();
      } else if (da.kind == Dim::UNDEF || db.kind == Dim::UNDEF) {
        // a known extent other than 1 fixes the output even if the partner is unknown
        if (da.known() && !is1(da) && da.e.is_const()) o.dims[i] = da;
        else if (db.known() && !is1(db) && db.e.is_const()) o.dims[i] = db;
        else o.dims[i] = Dim();
      } else if (da == db) o.dims[i] = da;
      else if (is1(db)) o.dims[i] = da;
      else if (is1(da)) o.dims[i] = db;
      else if (da.e.is_const() && db.e.is_const()) {
        fail(E_SHAPE_CONFLICT, who + ": cannot broadcast " + e_str(g.cx, da.e) + " with " + e_str(g.cx, db.e));
      } else {
        // neither provably 1 nor provably equal: both fused versions would be needed
        if (unresolved) ++*unresolved;
        add_bcast_assert(da.e, db.e, who + ": broadcast of " + e_str(g.cx, da.e) + " with " + e_str(g.cx, db.e));
        o.dims[i] = Dim::val(e_max(g.cx, da.e, db.e));
      }
    }
    return o;
  }

  // integer arithmetic on tracked values (shape tensors)
  ValueVal vbinary(const std::string& op, const ValueVal& a, const ValueVal& b) {
    ValueVal o;
    if (a.kind == ValueVal::NAC || b.kind == ValueVal::NAC) { o.kind = ValueVal::NAC; return o; }
    if (a.kind != ValueVal::KNOWN || b.kind != ValueVal::KNOWN) return o;
    size_t n = std::max(a.elems.size(), b.elems.size());
    if ((a.elems.size() != n && a.elems.size() != 1) || (b.elems.size() != n && b.elems.size() != 1)) { o.kind = ValueVal::NAC; return o; }
    o.kind = ValueVal::KNOWN;
    o.elems.resize(n);
    for (size_t i = 0; i < n; ++i) {
      const Dim& x = a.elems[a.elems.size() == 1 ? 0 : i];
      const Dim& y = b.elems[b.elems.size() == 1 ? 0 : i];
      if (!x.known() || !y.known()) { o.elems[i] = (x.kind == Dim::NAC || y.kind == Dim::NAC) ? Dim::nac() : Dim(); continue; }
      if (op == "Add") o.elems[i] = Dim::val(x.e + y.e);
      else if (op == "Sub") o.elems[i] = Dim::val(x.e - y.e);
      else if (op == "Mul") o.elems[i] = Dim::val(x.e * y.e);
      else if (op == "Div") o.elems[i] = Dim::val(e_floordiv(g.cx, x.e, y.e));
      else o.elems[i] = Dim::nac();
    }
    return o;
  }

  bool is_int_tensor(int t) const { return g.tensors[t].dtype == DType::I64; }

  Expr numel(const ShapeVal& s) {
    Expr p(1);
    for (auto& d : s.dims) p = p * d.e;
    return p;
  }

  // ---------------------------------------------------------------- forward Update functions
  bool forward(int nid) {
    Node& n = g.nodes[nid];
    bool need = false;
    for (int o : n.outs) {
      const Tensor& T = g.tensors[o];
      if (T.S.any_undef()) need = true;
      if (is_int_tensor(o) && T.V.kind == ValueVal::UNDEF) need = true;
      if (T.V.kind == ValueVal::KNOWN && !T.V.all_known()) need = true;
    }
    if (!need) return false;  // outputs are not in undef (Algorithm 1, forward_transfer)
    bool ch = false;
    const std::string& op = n.op;
    auto in = [&](int i) { return n.ins[i]; };
    auto out = [&](int i) { return n.outs[i]; };
    auto nin = n.ins.size();

    if (op == "Shape") {                                   // F^fs_ISDO / F^fv_ISDO
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = DType::I64;
      if (x.rank >= 0) {
        ShapeVal s; s.rank = 1; s.dims = {Dim::c(x.rank)};
        ch |= refine_shape(out(0), s);
        ValueVal v; v.kind = ValueVal::KNOWN; v.elems = x.dims;
        ch |= refine_value(out(0), v);
      } else if (x.rank == RANK_NAC) {
        ShapeVal s; s.rank = 1; s.dims = {Dim::nac()};
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "ConstantOfShape") {
      const ValueVal& v = V(in(0));
      if (v.kind == ValueVal::KNOWN) { ShapeVal s; s.rank = static_cast<int>(v.elems.size()); s.dims = v.elems; ch |= refine_shape(out(0), s); }
      else if (v.kind == ValueVal::NAC) { ShapeVal s; s.rank = RANK_NAC; ch |= refine_shape(out(0), s); }
    } else if (op == "Add" || op == "Sub" || op == "Mul" || op == "Div" || op == "Greater") {  // F^fs_ISDOS
      int unres = 0;
      ShapeVal s = bcast(S(in(0)), S(in(1)), op + " -> " + g.tensors[out(0)].name, &unres);
      n.attrs["unresolved_bcast"] = std::to_string(unres);
      ch |= refine_shape(out(0), s);
      if (op == "Greater") g.tensors[out(0)].dtype = DType::BOOL;
      else if (is_int_tensor(in(0)) && is_int_tensor(in(1))) {
        g.tensors[out(0)].dtype = DType::I64;
        ch |= refine_value(out(0), vbinary(op, V(in(0)), V(in(1))));
      } else g.tensors[out(0)].dtype = g.tensors[in(0)].kind == TKind::FCONST ? g.tensors[in(1)].dtype : g.tensors[in(0)].dtype;
    } else if (op == "Relu" || op == "Sigmoid" || op == "Gelu" || op == "Softmax" || op == "LayerNormalization" ||
               op == "Round" || op == "Cast" || op == "ToChannelsLast" || op == "FromChannelsLast") {
      ch |= refine_shape(out(0), S(in(0)));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (op == "Cast") {
        DType dt;
        if (parse_dtype(n.attr_s("to", "f32"), &dt)) g.tensors[out(0)].dtype = dt;
        if (is_int_tensor(in(0)) && dt == DType::I64) ch |= refine_value(out(0), V(in(0)));
      }
    } else if (op == "MatMul") {
      const ShapeVal &a = S(in(0)), &b = S(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (a.rank >= 2 && b.rank >= 2) {
        ShapeVal ba, bb;
        ba.rank = a.rank - 2; ba.dims.assign(a.dims.begin(), a.dims.end() - 2);
        bb.rank = b.rank - 2; bb.dims.assign(b.dims.begin(), b.dims.end() - 2);
        ShapeVal s = bcast(ba, bb, "MatMul batch", nullptr);
        s.dims.push_back(a.dims[a.rank - 2]);
        s.dims.push_back(b.dims[b.rank - 1]);
        s.rank += 2;
        ch |= refine_shape(out(0), s);
      } else if (a.rank == RANK_NAC || b.rank == RANK_NAC) { ShapeVal s; s.rank = RANK_NAC; ch |= refine_shape(out(0), s); }
      else if (a.rank >= 0 && b.rank >= 0) fail(E_RANK_MISMATCH, "MatMul needs rank >= 2");
    } else if (op == "Conv") {
      const ShapeVal &x = S(in(0)), &w = S(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (x.rank == 4 && w.rank == 4 && w.fully_known()) {
        int64_t s_ = n.attr_i("stride", 1), p = n.attr_i("pad", 0);
        ShapeVal s; s.rank = 4; s.dims.resize(4);
        s.dims[0] = x.dims[0];
        s.dims[1] = w.dims[0];
        for (int d = 2; d < 4; ++d) {
          if (!x.dims[d].known()) { s.dims[d] = x.dims[d]; continue; }
          // floor((in + 2p - k) / s) + 1; for k=3,p=1,s=1 this simplifies to exactly `in`
          Expr num = x.dims[d].e + Expr(2 * p) - w.dims[d].e;
          s.dims[d] = Dim::val(e_floordiv(g.cx, num, Expr(s_)) + Expr(1));
        }
        ch |= refine_shape(out(0), s);
      } else if (x.rank >= 0 && x.rank != 4) fail(E_RANK_MISMATCH, "Conv needs NCHW input");
    } else if (op == "GlobalAveragePool") {
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (x.rank == 4) { ShapeVal s; s.rank = 4; s.dims = {x.dims[0], x.dims[1], Dim::c(1), Dim::c(1)}; ch |= refine_shape(out(0), s); }
      else if (x.rank >= 0) fail(E_RANK_MISMATCH, "GlobalAveragePool needs NCHW input");
    } else if (op == "ReduceSumSquare" || op == "ReduceMean" || op == "ReduceSum") {
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (x.rank >= 1) {
        int ax = norm_axis(n.attr_i("axis", -1), x.rank);
        ShapeVal s;
        for (int i = 0; i < x.rank; ++i) {
          if (i == ax) { if (n.attr_i("keepdims", 1)) s.dims.push_back(Dim::c(1)); }
          else s.dims.push_back(x.dims[i]);
        }
        s.rank = static_cast<int>(s.dims.size());
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "Concat") {
      bool all = true;
      for (size_t i = 0; i < nin; ++i) if (S(in(i)).rank < 0) all = false;
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (all) {
        int rank = S(in(0)).rank;
        int ax = norm_axis(n.attr_i("axis", 0), rank);
        ShapeVal s = S(in(0));
        Dim sum = Dim::c(0);
        for (size_t i = 0; i < nin; ++i) {
          const ShapeVal& x = S(in(i));
          if (x.rank != rank) { fail(E_RANK_MISMATCH, "Concat ranks differ"); return ch; }
          const Dim& d = x.dims[ax];
          if (sum.kind == Dim::VAL && d.known()) sum = Dim::val(sum.e + d.e);
          else sum = (d.kind == Dim::NAC || sum.kind == Dim::NAC) ? Dim::nac() : Dim();
          for (int k = 0; k < rank; ++k) if (k != ax) s.dims[k] = meet(s.dims[k], x.dims[k]);
        }
        s.dims[ax] = sum;
        ch |= refine_shape(out(0), s);
        if (is_int_tensor(in(0)) && rank == 1) {
          ValueVal v; v.kind = ValueVal::KNOWN;
          for (size_t i = 0; i < nin; ++i) {
            const ValueVal& x = V(in(i));
            if (x.kind == ValueVal::NAC) { v.kind = ValueVal::NAC; break; }
            if (x.kind != ValueVal::KNOWN) { v.kind = ValueVal::UNDEF; break; }
            v.elems.insert(v.elems.end(), x.elems.begin(), x.elems.end());
          }
          if (v.kind != ValueVal::KNOWN) v.elems.clear();
          ch |= refine_value(out(0), v);
        }
      }
    } else if (op == "Gather") {
      const ShapeVal &d = S(in(0)), &ix = S(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (d.rank >= 1 && ix.rank >= 0) {
        int ax = norm_axis(n.attr_i("axis", 0), d.rank);
        ShapeVal s;
        s.dims.insert(s.dims.end(), d.dims.begin(), d.dims.begin() + ax);
        s.dims.insert(s.dims.end(), ix.dims.begin(), ix.dims.end());
        s.dims.insert(s.dims.end(), d.dims.begin() + ax + 1, d.dims.end());
        s.rank = static_cast<int>(s.dims.size());
        ch |= refine_shape(out(0), s);
        // value of a shape tensor picked by constant indices (how "N" is extracted from Shape)
        if (is_int_tensor(in(0)) && d.rank == 1) {
          const ValueVal &dv = V(in(0)), &iv = V(in(1));
          if (dv.kind == ValueVal::KNOWN && iv.all_known()) {
            ValueVal v; v.kind = ValueVal::KNOWN;
            bool ok = true;
            for (auto& e : iv.elems) {
              if (!e.e.is_const()) { ok = false; break; }
              int64_t k = e.e.const_value();
              if (k < 0) k += static_cast<int64_t>(dv.elems.size());
              if (k < 0 || k >= static_cast<int64_t>(dv.elems.size())) { fail(E_BAD_DIM, "Gather index out of range"); return ch; }
              v.elems.push_back(dv.elems[k]);
            }
            if (ok) ch |= refine_value(out(0), v);
          } else if (dv.kind == ValueVal::NAC || iv.kind == ValueVal::NAC) {
            ValueVal v; v.kind = ValueVal::NAC; ch |= refine_value(out(0), v);
          }
        }
      }
    } else if (op == "Transpose") {
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      std::vector<int64_t> perm = n.attr_list("perm");
      if (x.rank >= 0) {
        if (static_cast<int>(perm.size()) != x.rank) { fail(E_RANK_MISMATCH, "Transpose perm length"); return ch; }
        ShapeVal s; s.rank = x.rank; s.dims.resize(x.rank);
        for (int i = 0; i < x.rank; ++i) s.dims[i] = x.dims[perm[i]];
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "Reshape") {                          // F^fs_ISVDOS
      const ShapeVal& x = S(in(0));
      const ValueVal& sv = V(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (sv.kind == ValueVal::NAC) {
        ShapeVal s;
        const ShapeVal& ss = S(in(1));
        if (ss.rank == 1 && ss.dims[0].known() && ss.dims[0].e.is_const()) { s.rank = static_cast<int>(ss.dims[0].e.const_value()); s.dims.assign(s.rank, Dim::nac()); }
        else s.rank = RANK_NAC;
        ch |= refine_shape(out(0), s);
      } else if (sv.all_known() && x.rank >= 0) {
        ShapeVal s; s.rank = static_cast<int>(sv.elems.size()); s.dims.resize(s.rank);
        int minus1 = -1;
        Expr prod(1);
        bool ok = true;
        for (int i = 0; i < s.rank; ++i) {
          const Expr& e = sv.elems[i].e;
          if (e.is_const() && e.const_value() == -1) { if (minus1 >= 0) { fail(E_BAD_DIM, "Reshape: two -1"); return ch; } minus1 = i; continue; }
          if (e.is_const() && e.const_value() == 0) {
            if (i >= x.rank) { fail(E_BAD_DIM, "Reshape: 0 beyond input rank"); return ch; }
            s.dims[i] = x.dims[i];
          } else s.dims[i] = Dim::val(e);
          if (!s.dims[i].known()) ok = false; else prod = prod * s.dims[i].e;
        }
        if (minus1 >= 0) {
          if (ok && x.fully_known()) {
            bool dok;
            Expr q = e_exact_div(numel(x), prod, &dok);
            s.dims[minus1] = Dim::val(dok ? q : e_floordiv(g.cx, numel(x), prod));
          } else s.dims[minus1] = Dim();
        } else if (ok && x.fully_known()) {
          add_assert(numel(x), prod, "Reshape numel of " + g.tensors[out(0)].name);
        }
        ch |= refine_shape(out(0), s);
        if (is_int_tensor(in(0))) ch |= refine_value(out(0), V(in(0)));
      }
    } else if (op == "Slice") {
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (nin < 3) { fail(E_INVALID_ARG, "Slice needs data, starts, ends"); return ch; }
      const ValueVal &st_ = V(in(1)), &en = V(in(2));
      bool nacv = st_.kind == ValueVal::NAC || en.kind == ValueVal::NAC;
      if (x.rank >= 0 && nacv) {
        ShapeVal s = x;
        for (auto& d : s.dims) d = Dim::nac();
        ch |= refine_shape(out(0), s);
      } else if (x.rank >= 0 && st_.all_known() && en.all_known()) {
        size_t k = st_.elems.size();
        std::vector<int64_t> axes(k), steps(k, 1);
        for (size_t i = 0; i < k; ++i) axes[i] = static_cast<int64_t>(i);
        if (nin > 3) { const ValueVal& av = V(in(3)); if (!av.all_known()) return ch; for (size_t i = 0; i < k; ++i) axes[i] = av.elems[i].e.const_value(); }
        if (nin > 4) { const ValueVal& sv = V(in(4)); if (!sv.all_known()) return ch; for (size_t i = 0; i < k; ++i) steps[i] = sv.elems[i].e.const_value(); }
        ShapeVal s = x;
        ValueVal vout;
        for (size_t i = 0; i < k; ++i) {
          int ax = norm_axis(axes[i], x.rank);
          const Dim& d = x.dims[ax];
          if (!d.known()) { s.dims[ax] = d; continue; }
          Expr b = st_.elems[i].e, e = en.elems[i].e;
          if (steps[i] <= 0) { fail(E_UNSUPPORTED_OP, "Slice: non-positive step"); return ch; }
          auto clampc = [&](Expr v) {  // negative constants count from the end
            if (v.is_const() && v.const_value() < 0) v = v + d.e;
            return v;
          };
          b = clampc(b); e = clampc(e);
          if (b.is_const() && e.is_const() && d.e.is_const()) {
            int64_t D = d.e.const_value(), bb = std::min(std::max<int64_t>(b.const_value(), 0), D), ee = std::min(std::max<int64_t>(e.const_value(), 0), D);
            int64_t len = ee > bb ? (ee - bb + steps[i] - 1) / steps[i] : 0;
            s.dims[ax] = Dim::c(len);
            n.attrs["_start" + std::to_string(ax)] = std::to_string(bb);
          } else {
            Expr ee = e_min(g.cx, e, d.e);
            s.dims[ax] = Dim::val(e_ceildiv(g.cx, ee - b, Expr(steps[i])));
            if (b.is_const()) n.attrs["_start" + std::to_string(ax)] = std::to_string(b.const_value());
          }
          n.attrs["_step" + std::to_string(ax)] = std::to_string(steps[i]);
        }
        ch |= refine_shape(out(0), s);
        // Slice of a shape tensor: evaluates on the value map
        if (is_int_tensor(in(0)) && x.rank == 1 && V(in(0)).kind == ValueVal::KNOWN && s.dims[0].known() && s.dims[0].e.is_const()) {
          int64_t b = std::strtoll(n.attr_s("_start0", "0").c_str(), nullptr, 10);
          ValueVal v; v.kind = ValueVal::KNOWN;
          for (int64_t j = 0; j < s.dims[0].e.const_value(); ++j) v.elems.push_back(V(in(0)).elems[b + j * steps[0]]);
          ch |= refine_value(out(0), v);
        }
      }
    } else if (op == "TopK") {
      const ShapeVal& x = S(in(0));
      const ValueVal& kv = V(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (n.outs.size() > 1) g.tensors[out(1)].dtype = DType::I64;
      if (x.rank >= 1 && kv.kind != ValueVal::UNDEF) {
        int ax = norm_axis(n.attr_i("axis", -1), x.rank);
        ShapeVal s = x;
        s.dims[ax] = (kv.kind == ValueVal::KNOWN && kv.elems.size() == 1) ? kv.elems[0] : Dim::nac();
        for (int o : n.outs) ch |= refine_shape(o, s);
      }
    } else if (op == "Range") {
      g.tensors[out(0)].dtype = DType::I64;
      const ValueVal &a = V(in(0)), &b = V(in(1)), &c = V(in(2));
      if (a.all_known() && b.all_known() && c.all_known()) {
        ShapeVal s; s.rank = 1;
        Expr len = e_max(g.cx, e_ceildiv(g.cx, b.elems[0].e - a.elems[0].e, c.elems[0].e), Expr(0));
        s.dims = {Dim::val(len)};
        ch |= refine_shape(out(0), s);
        if (len.is_const() && len.const_value() <= 16 && a.elems[0].e.is_const() && c.elems[0].e.is_const()) {
          ValueVal v; v.kind = ValueVal::KNOWN;
          for (int64_t i = 0; i < len.const_value(); ++i) v.elems.push_back(Dim::c(a.elems[0].e.const_value() + i * c.elems[0].e.const_value()));
          ch |= refine_value(out(0), v);
        }
      } else if (a.kind == ValueVal::NAC || b.kind == ValueVal::NAC || c.kind == ValueVal::NAC) {
        ShapeVal s; s.rank = 1; s.dims = {Dim::nac()};
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "NonZero") {                          // F^fs_EDO: rank fixed, count known only after execution
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = DType::I64;
      if (x.rank >= 0) {
        ShapeVal s; s.rank = 2;
        int sym = g.cx.symbol("nnz(" + g.tensors[in(0)].name + ")", 0, INT64_MAX, true);
        if (x.fully_known()) g.cx.atoms[sym].hi_expr = std::make_shared<Expr>(numel(x));
        s.dims = {Dim::c(x.rank), Dim::val(Expr::atom(sym))};
        ch |= refine_shape(out(0), s);
        ValueVal v; v.kind = ValueVal::NAC;
        ch |= refine_value(out(0), v);
      }
    } else if (op == "EyeLike" || op == "GroupNormalization") {    // output shape = shape of the first input
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (S(in(0)).rank != RANK_UNDEF) ch |= refine_shape(out(0), S(in(0)));
    } else if (op == "AveragePool" || op == "MaxPool") {           // F^fs_ISDOS: windows over H, W
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (x.rank == 4) {
        const int64_t k = n.attr_i("kernel", 2), s_ = n.attr_i("stride", k), p = n.attr_i("pad", 0);
        ShapeVal s; s.rank = 4; s.dims = {x.dims[0], x.dims[1], x.dims[2], x.dims[3]};
        for (int d = 2; d < 4; ++d)
          if (x.dims[d].known()) s.dims[d] = Dim::val(e_floordiv(g.cx, x.dims[d].e + Expr(2 * p - k), Expr(s_)) + Expr(1));
        ch |= refine_shape(out(0), s);
      } else if (x.rank >= 0) fail(E_RANK_MISMATCH, op + " needs NCHW input");
    } else if (op == "Expand") {                                   // F^fs_ISVDOS: broadcast against the VALUE of the shape input
      const ValueVal& v = V(in(1));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (v.kind == ValueVal::KNOWN) {
        ShapeVal t; t.rank = static_cast<int>(v.elems.size()); t.dims = v.elems;
        int unres = 0;
        ShapeVal s = bcast(S(in(0)), t, "Expand -> " + g.tensors[out(0)].name, &unres);
        n.attrs["unresolved_bcast"] = std::to_string(unres);
        ch |= refine_shape(out(0), s);
      } else if (v.kind == ValueVal::NAC) { ShapeVal s; s.rank = RANK_NAC; ch |= refine_shape(out(0), s); }
    } else if (op == "Resize" || op == "Upsample") {                // F^fs_ISVDOS: sizes input (values) or integer scales attribute
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      const std::vector<int64_t> sc = n.attr_list("scales");
      if (n.ins.size() > 1) {
        const ValueVal& v = V(in(1));
        if (v.kind == ValueVal::KNOWN) {
          ShapeVal s; s.rank = static_cast<int>(v.elems.size()); s.dims = v.elems;
          if (x.rank >= 0 && x.rank != s.rank) fail(E_RANK_MISMATCH, op + ": sizes must have the input's rank");
          else ch |= refine_shape(out(0), s);
        } else if (v.kind == ValueVal::NAC && x.rank >= 0) {
          ShapeVal s; s.rank = x.rank; s.dims.assign(x.rank, Dim::nac());
          ch |= refine_shape(out(0), s);
        }
      } else if (x.rank >= 0) {
        if (static_cast<int>(sc.size()) != x.rank) fail(E_BAD_DIM, op + ": scales must list one integer per axis");
        else {
          ShapeVal s; s.rank = x.rank; s.dims.resize(x.rank);
          for (int d = 0; d < x.rank; ++d) s.dims[d] = x.dims[d].known() ? Dim::val(x.dims[d].e * Expr(sc[d])) : x.dims[d];
          ch |= refine_shape(out(0), s);
        }
      }
    } else if (op == "OneHot") {                                    // F^fs_ISVDOS: indices shape + [depth value]
      const ShapeVal& x = S(in(0));
      const ValueVal& v = V(in(1));
      if (x.rank >= 0 && v.kind == ValueVal::KNOWN && v.elems.size() == 1) {
        ShapeVal s = x; s.rank = x.rank + 1; s.dims.push_back(v.elems[0]);
        ch |= refine_shape(out(0), s);
      } else if (x.rank >= 0 && v.kind == ValueVal::NAC) {
        ShapeVal s = x; s.rank = x.rank + 1; s.dims.push_back(Dim::nac());
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "MaxUnpool") {                                 // F^fs_ISVDOS: output_shape input (values), else from the window
      const ShapeVal& x = S(in(0));
      g.tensors[out(0)].dtype = g.tensors[in(0)].dtype;
      if (n.ins.size() > 2) {
        const ValueVal& v = V(in(2));
        if (v.kind == ValueVal::KNOWN) { ShapeVal s; s.rank = static_cast<int>(v.elems.size()); s.dims = v.elems; ch |= refine_shape(out(0), s); }
        else if (v.kind == ValueVal::NAC && x.rank >= 0) { ShapeVal s; s.rank = x.rank; s.dims.assign(x.rank, Dim::nac()); ch |= refine_shape(out(0), s); }
      } else if (x.rank == 4) {
        const int64_t k = n.attr_i("kernel", 2), s_ = n.attr_i("stride", k), p = n.attr_i("pad", 0);
        ShapeVal s; s.rank = 4; s.dims = {x.dims[0], x.dims[1], x.dims[2], x.dims[3]};
        for (int d = 2; d < 4; ++d)
          if (x.dims[d].known()) s.dims[d] = Dim::val((x.dims[d].e - Expr(1)) * Expr(s_) + Expr(k - 2 * p));
        ch |= refine_shape(out(0), s);
      }
    } else if (op == "NonMaxSuppression") {                         // F^fs_EDO: [selected, 3], the count known only after execution
      const ShapeVal& sc = S(in(1));                                // scores [batch, classes, boxes]
      g.tensors[out(0)].dtype = DType::I64;
      if (sc.rank >= 0) {
        int sym = g.cx.symbol("nms(" + g.tensors[in(1)].name + ")", 0, INT64_MAX, true);
        if (sc.fully_known()) g.cx.atoms[sym].hi_expr = std::make_shared<Expr>(numel(sc));
        ShapeVal s; s.rank = 2; s.dims = {Dim::val(Expr::atom(sym)), Dim::c(3)};
        ch |= refine_shape(out(0), s);
        ValueVal v; v.kind = ValueVal::NAC;
        ch |= refine_value(out(0), v);
      }
    } else {
      fail(E_UNSUPPORTED_OP, "no transfer function for " + op);
    }
    return ch;
  }

  // Switch (execution determined): the two branch tensors split the leading (sample) dim by a
  // run-time count; the count of one gate is one runtime symbol shared by every Switch on it.
  bool switch_transfer(int nid) {
    Node& n = g.nodes[nid];
    const ShapeVal& x = S(n.ins[0]);
    if (x.rank < 1 || !x.dims[0].known()) return false;
    int sym = g.cx.symbol("count(" + g.tensors[n.ins[1]].name + ")", 0, INT64_MAX, true);
    g.cx.atoms[sym].hi_expr = std::make_shared<Expr>(x.dims[0].e);
    ShapeVal a = x, b = x;
    a.dims[0] = Dim::val(Expr::atom(sym));
    b.dims[0] = Dim::val(x.dims[0].e - Expr::atom(sym));
    bool ch = false;
    for (int o : n.outs) g.tensors[o].dtype = g.tensors[n.ins[0]].dtype;
    ch |= refine_shape(n.outs[0], a);
    if (n.outs.size() > 1) ch |= refine_shape(n.outs[1], b);
    return ch;
  }

  // Merge (Section 4.1): meet of the S-maps arriving at Combine; the regrouped sample dim is the
  // sum of the branches' sample dims (canonically the original batch extent).
  bool merge(int nid) {
    Node& n = g.nodes[nid];
    const ShapeVal &a = S(n.ins[0]), &b = S(n.ins[1]);
    if (a.rank < 1 || b.rank < 1) return false;
    if (a.rank != b.rank) { fail(E_RANK_MISMATCH, "Combine branch ranks differ"); return false; }
    ShapeVal s; s.rank = a.rank; s.dims.resize(a.rank);
    for (int i = 1; i < a.rank; ++i) s.dims[i] = meet(a.dims[i], b.dims[i]);
    if (a.dims[0].known() && b.dims[0].known()) s.dims[0] = Dim::val(a.dims[0].e + b.dims[0].e);
    else s.dims[0] = (a.dims[0].kind == Dim::NAC || b.dims[0].kind == Dim::NAC) ? Dim::nac() : Dim();
    g.tensors[n.outs[0]].dtype = g.tensors[n.ins[0]].dtype;
    // a meet that yields nac must override an earlier optimistic value
    Tensor& T = g.tensors[n.outs[0]];
    bool ch = false;
    if (T.S.rank == RANK_UNDEF) { T.S = s; return true; }
    for (int i = 0; i < s.rank; ++i) {
      Dim m = meet(T.S.dims[i], s.dims[i]);
      if (m != T.S.dims[i]) { T.S.dims[i] = m; ch = true; }
    }
    return ch;
  }

  // ---------------------------------------------------------------- backward Update functions
  // Only refinements that are unambiguous are applied: same-shape operators, the contracted dim of
  // MatMul, Transpose, Conv channels, the input of Shape from the value of its output, the one unknown
  // extent of a Reshape input from the element count, the one unknown Concat operand.  Broadcasting operators
  // give a set {1, d} per dim in general (Section 3), which the lattice cannot hold: they propagate the rank
  // when it is certain, and an extent where the partner's is the constant 1.
  bool backward(int nid, int pred_tensor) {
    const Tensor& P = g.tensors[pred_tensor];
    if (!P.S.any_undef()) return false;
    Node& n = g.nodes[nid];
    const std::string& op = n.op;
    bool ch = false;
    if ((op == "Relu" || op == "Sigmoid" || op == "Gelu" || op == "Softmax" || op == "LayerNormalization" || op == "Round" || op == "Cast" ||
         op == "ToChannelsLast" || op == "FromChannelsLast") &&
        pred_tensor == n.ins[0]) {
      ch |= refine_shape(pred_tensor, S(n.outs[0]));
    } else if (op == "MatMul") {
      const ShapeVal &a = S(n.ins[0]), &b = S(n.ins[1]), &o = S(n.outs[0]);
      if (pred_tensor == n.ins[0] && a.rank >= 2) {
        ShapeVal s = a;
        if (b.rank >= 2) s.dims[a.rank - 1] = b.dims[b.rank - 2];
        if (o.rank >= 2) s.dims[a.rank - 2] = o.dims[o.rank - 2];
        ch |= refine_shape(pred_tensor, s);
      } else if (pred_tensor == n.ins[1] && b.rank >= 2) {
        ShapeVal s = b;
        if (a.rank >= 2) s.dims[b.rank - 2] = a.dims[a.rank - 1];
        if (o.rank >= 2) s.dims[b.rank - 1] = o.dims[o.rank - 1];
        ch |= refine_shape(pred_tensor, s);
      }
    } else if (op == "Transpose") {
      const ShapeVal& o = S(n.outs[0]);
      std::vector<int64_t> perm = n.attr_list("perm");
      if (o.rank >= 0 && static_cast<int>(perm.size()) == o.rank) {
        ShapeVal s; s.rank = o.rank; s.dims.resize(o.rank);
        for (int i = 0; i < o.rank; ++i) s.dims[perm[i]] = o.dims[i];
        ch |= refine_shape(pred_tensor, s);
      }
    } else if (op == "Conv" && pred_tensor == n.ins[0]) {
      const ShapeVal &w = S(n.ins[1]), &o = S(n.outs[0]);
      if (w.rank == 4) {
        ShapeVal s; s.rank = 4; s.dims.assign(4, Dim());
        s.dims[1] = w.dims[1];
        if (o.rank == 4) s.dims[0] = o.dims[0];
        ch |= refine_shape(pred_tensor, s);
      }
    } else if (op == "Add" || op == "Sub" || op == "Mul" || op == "Div") {
      const ShapeVal& o = S(n.outs[0]);
      int other = pred_tensor == n.ins[0] ? n.ins[1] : n.ins[0];
      const ShapeVal& q = S(other);
      if (P.S.rank == RANK_UNDEF) {
        // rank certain only if the partner has lower rank than the output
        if (o.rank >= 0 && q.rank >= 0 && q.rank < o.rank) {
          ShapeVal s; s.rank = o.rank; s.dims.assign(o.rank, Dim());
          ch |= refine_shape(pred_tensor, s);
        }
      } else if (o.rank >= 0 && q.rank >= 0 && P.S.rank == o.rank) {
        // broadcasting leaves {1, d} for an extent in general; where the PARTNER's extent is the constant 1 (or the
        // partner has no such dim) and the output's is another value, this operand must carry the output's extent
        ShapeVal s = P.S;
        for (int i = 0; i < o.rank; ++i) {
          const int qi = i - (o.rank - q.rank);
          const bool partner_one = qi < 0 || (q.dims[qi].known() && q.dims[qi].e.is_const() && q.dims[qi].e.const_value() == 1);
          const bool out_not_one = o.dims[i].known() && !(o.dims[i].e.is_const() && o.dims[i].e.const_value() == 1);
          if (s.dims[i].kind == Dim::UNDEF && partner_one && out_not_one) s.dims[i] = o.dims[i];
        }
        ch |= refine_shape(pred_tensor, s);
      }
    } else if (op == "Shape" && pred_tensor == n.ins[0]) {
      // F^bs of the shape-determined-output class: the VALUE of Shape's output is its input's shape
      const ValueVal& v = V(n.outs[0]);
      if (v.kind == ValueVal::KNOWN) {
        ShapeVal s; s.rank = static_cast<int>(v.elems.size()); s.dims = v.elems;
        ch |= refine_shape(pred_tensor, s);
      } else if (S(n.outs[0]).rank == 1 && S(n.outs[0]).dims[0].known() && S(n.outs[0]).dims[0].e.is_const() && P.S.rank == RANK_UNDEF) {
        ShapeVal s; s.rank = static_cast<int>(S(n.outs[0]).dims[0].e.const_value()); s.dims.assign(s.rank, Dim());
        ch |= refine_shape(pred_tensor, s);
      }
    } else if (op == "Reshape" && pred_tensor == n.ins[0]) {
      // one unknown input extent follows from the element count of a fully known output
      const ShapeVal& o = S(n.outs[0]);
      if (o.fully_known() && P.S.rank >= 1) {
        int unknown = -1, n_unknown = 0;
        Expr known_prod(1), total(1);
        for (int i = 0; i < P.S.rank; ++i) {
          if (P.S.dims[i].kind == Dim::UNDEF) { unknown = i; ++n_unknown; }
          else if (P.S.dims[i].known()) known_prod = known_prod * P.S.dims[i].e;
          else n_unknown = 99;
        }
        for (auto& d : o.dims) total = total * d.e;
        bool okq = false;
        const Expr quot = n_unknown == 1 ? e_exact_div(total, known_prod, &okq) : Expr();
        if (n_unknown == 1 && okq) {
          ShapeVal s = P.S;
          s.dims[unknown] = Dim::val(quot);
          ch |= refine_shape(pred_tensor, s);
        }
      }
    } else if (op == "Concat") {
      // the extents off the axis equal the output's; on the axis the one unknown operand takes what is left
      const ShapeVal& o = S(n.outs[0]);
      if (o.rank >= 1 && (P.S.rank == o.rank || P.S.rank == RANK_UNDEF)) {
        const int ax = norm_axis(n.attr_i("axis", 0), o.rank);
        ShapeVal s; s.rank = o.rank; s.dims.assign(o.rank, Dim());
        if (P.S.rank == o.rank) s = P.S;
        for (int i = 0; i < o.rank; ++i) if (i != ax && s.dims[i].kind == Dim::UNDEF) s.dims[i] = o.dims[i];
        if (s.dims[ax].kind == Dim::UNDEF && o.dims[ax].known()) {
          Expr rest = o.dims[ax].e;
          bool ok = true;
          int mine = 0;
          for (int in_t : n.ins) {
            if (in_t == pred_tensor) { ++mine; continue; }
            const ShapeVal& x = S(in_t);
            if (x.rank != o.rank || !x.dims[ax].known()) { ok = false; break; }
            rest = rest - x.dims[ax].e;
          }
          if (ok && mine == 1) s.dims[ax] = Dim::val(rest);
        }
        ch |= refine_shape(pred_tensor, s);
      }
    }
    return ch;
  }

  // Algorithm 1 step 3: a Shape node whose input rank is known gets a symbolic value; extents that
  // no transfer function could determine are named as fresh symbolic constants, on the input too.
  bool isdo_symbolic_value(int nid) {
    Node& n = g.nodes[nid];
    if (n.op != "Shape") return false;
    Tensor& X = g.tensors[n.ins[0]];
    if (X.S.rank < 0) return false;
    bool ch = false;
    for (int i = 0; i < X.S.rank; ++i) {
      if (X.S.dims[i].kind == Dim::UNDEF) {
        int sym = g.cx.symbol(X.name + ".d" + std::to_string(i), 0, INT64_MAX, false);
        g.user_syms.push_back(sym);
        X.S.dims[i] = Dim::val(Expr::atom(sym));
        ch = true;
      }
    }
    if (ch) {
      ValueVal v; v.kind = ValueVal::KNOWN; v.elems = X.S.dims;
      g.tensors[n.outs[0]].V = v;
    }
    return ch;
  }
};

void dfs_order(Graph& g) {
  // depth-first from the graph's sources in declaration order; reverse post-order
  size_t N = g.nodes.size();
  std::vector<char> seen(N, 0);
  std::vector<int> post;
  std::function<void(int)> visit = [&](int n) {
    if (seen[n]) return;
    seen[n] = 1;
    for (int o : g.nodes[n].outs)
      for (int c : g.tensors[o].consumers) visit(c);
    post.push_back(n);
  };
  // iterate in reverse so that the reversed post-order keeps declaration order among roots
  for (int n = static_cast<int>(N) - 1; n >= 0; --n) {
    bool root = true;
    for (int i : g.nodes[n].ins) if (g.tensors[i].producer >= 0) root = false;
    if (root) visit(n);
  }
  for (int n = static_cast<int>(N) - 1; n >= 0; --n) visit(n);
  g.order.assign(post.rbegin(), post.rend());
}

}  // namespace

Status rdp_analysis(Graph* gp, const std::vector<int>* order_override) {
  Graph& g = *gp;
  Rdp r(g);
  // Initialise: every produced tensor undef (already so); model inputs and constants keep their
  // declared shapes (set_model_input_shape).
  dfs_order(g);
  const std::vector<int>& order = order_override ? *order_override : g.order;
  g.rdp_sweeps = 0;
  bool changed;
  do {
    do {
      changed = false;
      for (int nid : order) {
        Node& n = g.nodes[nid];
        if (n.op == "Combine") { changed |= r.merge(nid); continue; }
        if (n.op == "Switch") { changed |= r.switch_transfer(nid); continue; }
        changed |= r.forward(nid);                          // 1: forward transfer to the current node
        for (int p : n.ins) changed |= r.backward(nid, p);  // 2: backward transfer to predecessors
        if (r.st != OK) return r.st;
      }
      if (++g.rdp_sweeps > 256) { g.err = "RDP did not converge"; return E_NOT_CONVERGED; }
    } while (changed);
    // 3: symbolic values for Input-Shape-Determined-Output nodes still lacking them
    for (int nid : order)
      if (g.nodes[nid].cls == DynClass::ISDO) changed |= r.isdo_symbolic_value(nid);
  } while (changed);

  // Effective class after constant propagation (Section 3, discussion): a shape-and-value
  // determined operator whose shape-determining values are all known behaves as shape determined.
  for (auto& n : g.nodes) {
    n.eff_cls = n.cls;
    if (n.cls == DynClass::ISVDOS) {
      bool all = n.ins.size() > 1;
      for (size_t i = 1; i < n.ins.size(); ++i) if (!g.tensors[n.ins[i]].V.all_known()) all = false;
      if (all) n.eff_cls = DynClass::ISDOS;
    }
  }
  return OK;
}

}  // namespace sod2
