// Extended computational graph (DAG + <Switch, Combine>), the RDP lattice and its S/V maps.
// Paper Section 3 (operator classes), Section 4.1 (domain, transfer functions, Algorithm 1).
#pragma once
#include <map>
#include <string>
#include <vector>

#include "expr.h"

namespace sod2 {

enum class DType { F32, BF16, I64, BOOL };
inline int dtype_size(DType t) { return t == DType::F32 ? 4 : t == DType::BF16 ? 2 : t == DType::I64 ? 8 : 1; }

// ---- lattice (Section 4.1): undef is top, nac is bottom, everything else is an expression.
// An execution-determined extent is an expression over a *runtime* symbol (bound once the
// producing operator has run, with a static upper bound); it reports as nac to the analysis.
struct Dim {
  enum Kind { UNDEF, VAL, NAC } kind = UNDEF;
  Expr e;
  static Dim val(const Expr& x) { Dim d; d.kind = VAL; d.e = x; return d; }
  static Dim c(int64_t v) { return val(Expr(v)); }
  static Dim nac() { Dim d; d.kind = NAC; return d; }
  bool known() const { return kind == VAL; }
  bool operator==(const Dim& o) const { return kind == o.kind && (kind != VAL || e == o.e); }
  bool operator!=(const Dim& o) const { return !(*this == o); }
};
Dim meet(const Dim& a, const Dim& b);

constexpr int RANK_UNDEF = -1, RANK_NAC = -2;
struct ShapeVal {            // S-map entry
  int rank = RANK_UNDEF;
  std::vector<Dim> dims;
  bool fully_known() const {
    if (rank < 0) return false;
    for (auto& d : dims) if (!d.known()) return false;
    return true;
  }
  bool any_undef() const {
    if (rank == RANK_UNDEF) return true;
    for (auto& d : dims) if (d.kind == Dim::UNDEF) return true;
    return false;
  }
};
struct ValueVal {            // V-map entry: tracked for integer tensors of at most 16 elements
  enum Kind { UNDEF, KNOWN, NAC } kind = UNDEF;
  std::vector<Dim> elems;    // row-major
  bool all_known() const {
    if (kind != KNOWN) return false;
    for (auto& d : elems) if (!d.known()) return false;
    return true;
  }
};

enum class DynClass { ISDO = 0, ISDOS = 1, ISVDOS = 2, EDO = 3 };
const char* dyn_class_name(DynClass c);
// Table 2 of the paper; returns false for an operator the table (and this library) does not know.
bool classify_op(const std::string& op, DynClass* out);

enum class TKind { INPUT, CONST, ICONST, FCONST, VALUE };

struct Tensor {
  std::string name;
  DType dtype = DType::F32;
  TKind kind = TKind::VALUE;
  ShapeVal S;
  ValueVal V;
  int producer = -1;
  int out_slot = 0;
  std::vector<int> consumers;
  std::vector<int64_t> idata;  // ICONST
  double fdata = 0;            // FCONST
  bool is_output = false;
  int io_index = -1;           // position among inputs / outputs
  const void* dev_ptr = nullptr;  // CONST: caller-owned device memory
  size_t dev_bytes = 0;
};

struct Node {
  std::string op;
  std::vector<int> ins, outs;
  std::map<std::string, std::string> attrs;
  DynClass cls = DynClass::ISDOS;      // Table 2
  DynClass eff_cls = DynClass::ISDOS;  // after constant propagation (Section 3, discussion)
  int group = -1, subgraph = 0;
  int64_t attr_i(const std::string& k, int64_t dflt) const;
  double attr_f(const std::string& k, double dflt) const;
  std::vector<int64_t> attr_list(const std::string& k) const;
  std::string attr_s(const std::string& k, const std::string& dflt) const;
};

struct Assertion {           // bind-time check produced when two inferences must agree
  Expr a, b;
  std::string what;
  int kind = 0;              // 0: a == b; 1: broadcast-compatible (a == b, or one of them is 1)
};

struct Graph {
  ExprCtx cx;
  std::vector<Tensor> tensors;
  std::vector<Node> nodes;
  std::map<std::string, int> tindex;
  std::vector<int> inputs, outputs, consts;
  std::vector<int> user_syms;          // atom ids of declared symbols, in declaration order
  std::vector<Assertion> asserts;
  std::vector<int> order;              // depth-first sorted nodes (Algorithm 1)
  int rdp_sweeps = 0;
  bool has_conv = false;               // convolution graph: rank-4 float intermediates are stored channels-last
  std::string err;

  int tensor(const std::string& n) const { auto it = tindex.find(n); return it == tindex.end() ? -1 : it->second; }
};

enum Status {
  OK = 0, E_INVALID_ARG, E_PARSE, E_UNSUPPORTED_OP, E_RANK_MISMATCH, E_NOT_CONVERGED, E_UNBOUND_SYMBOL, E_BAD_DIM,
  E_SHAPE_CONFLICT, E_ARENA_TOO_SMALL, E_MISALIGNED, E_CUDA, E_TIMEOUT, E_INTERNAL
};

Status parse_ir(const char* text, size_t len, Graph* g);
// Algorithm 1. `order_override` (optional) replaces the depth-first order; used to test that the
// fixpoint does not depend on the visiting order.
Status rdp_analysis(Graph* g, const std::vector<int>* order_override = nullptr);
std::string shape_str(const Graph& g, const ShapeVal& s);

}  // namespace sod2
