// Integer expression algebra for rank-and-dimension propagation.
// The analysis domain of the paper (Section 4.1) holds known constants, symbolic constants and
// "operation-inferred" constants, i.e. expressions over the former.  An Expr is a canonical
// polynomial with int64 coefficients over atoms; an atom is a symbol or an opaque non-linear node
// (floordiv, min, max) whose arguments are again canonical Exprs.  Two Exprs denote the same
// lattice value iff their canonical forms are structurally equal.
#pragma once
#include <cstdint>
#include <map>
#include <memory>
#include <string>
#include <utility>
#include <vector>

namespace sod2 {

struct Expr;
enum class AtomKind { SYM, FLOORDIV, MIN, MAX };

struct Atom {
  AtomKind kind;
  std::string name;            // SYM
  bool runtime = false;        // SYM: bound only after an execution-determined operator has run
  int64_t lo = 1, hi = INT64_MAX;  // SYM: declared range (hi is the static upper bound of a runtime symbol)
  std::shared_ptr<Expr> a, b;  // non-linear nodes
  std::shared_ptr<Expr> hi_expr;  // runtime SYM: upper bound as an expression (may be null)
  std::string key;
};

// Atom table of one graph.
struct ExprCtx {
  std::vector<Atom> atoms;
  std::map<std::string, int> index;
  int symbol(const std::string& name, int64_t lo = 1, int64_t hi = INT64_MAX, bool runtime = false);
  int find_symbol(const std::string& name) const;
  int intern(Atom&& a);
};

using Monomial = std::vector<std::pair<int, int>>;  // sorted (atom id, power)

struct Expr {
  std::map<Monomial, int64_t> terms;  // no zero coefficients

  Expr() {}
  explicit Expr(int64_t c) { if (c) terms[Monomial()] = c; }
  static Expr atom(int id) { Expr e; e.terms[Monomial{{id, 1}}] = 1; return e; }

  bool is_const() const { return terms.empty() || (terms.size() == 1 && terms.begin()->first.empty()); }
  int64_t const_value() const { return terms.empty() ? 0 : terms.begin()->second; }
  bool is_symbol() const {
    return terms.size() == 1 && terms.begin()->second == 1 && terms.begin()->first.size() == 1 &&
           terms.begin()->first[0].second == 1;
  }
  bool operator==(const Expr& o) const { return terms == o.terms; }
  bool operator!=(const Expr& o) const { return !(*this == o); }
};

Expr operator+(const Expr& a, const Expr& b);
Expr operator-(const Expr& a, const Expr& b);
Expr operator*(const Expr& a, const Expr& b);
Expr e_floordiv(ExprCtx& cx, const Expr& a, const Expr& b);
Expr e_ceildiv(ExprCtx& cx, const Expr& a, const Expr& b);
Expr e_min(ExprCtx& cx, const Expr& a, const Expr& b);
Expr e_max(ExprCtx& cx, const Expr& a, const Expr& b);
// Exact quotient a / b if b divides a as polynomials (monomial or constant divisor); ok=false otherwise.
Expr e_exact_div(const Expr& a, const Expr& b, bool* ok);

std::string e_str(const ExprCtx& cx, const Expr& e);
// Evaluate with atom values for symbols (vals[id], only read for SYM atoms). ok=false on an unbound
// symbol (value INT64_MIN) or a division by zero.
int64_t e_eval(const ExprCtx& cx, const Expr& e, const std::vector<int64_t>& vals, bool* ok);
// Values of EVERY atom (symbols as given in vals, non-linear atoms evaluated once, children first:
// atoms are interned after their arguments).  Atoms that cannot be evaluated get INT64_MIN.
void e_eval_atoms(const ExprCtx& cx, std::vector<int64_t>* vals);
// Evaluate with a complete atom table from e_eval_atoms (no recursion); ok=false if an atom is unknown.
int64_t e_eval_flat(const Expr& e, const std::vector<int64_t>& atom_vals, bool* ok);
bool e_has_runtime(const ExprCtx& cx, const Expr& e);
// Static upper bound of e using the symbols' declared ranges (all coefficients must be >= 0 and
// non-linear atoms monotone); ok=false if none can be derived.
int64_t e_upper(const ExprCtx& cx, const Expr& e, const std::vector<int64_t>& vals, bool* ok);

}  // namespace sod2
