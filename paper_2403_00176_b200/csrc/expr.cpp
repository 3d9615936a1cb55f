#include "expr.h"

#include <algorithm>
#include <sstream>

namespace sod2 {

int ExprCtx::intern(Atom&& a) {
  auto it = index.find(a.key);
  if (it != index.end()) return it->second;
  int id = static_cast<int>(atoms.size());
  index[a.key] = id;
  atoms.push_back(std::move(a));
  return id;
}

int ExprCtx::symbol(const std::string& name, int64_t lo, int64_t hi, bool runtime) {
  Atom a;
  a.kind = AtomKind::SYM;
  a.name = name;
  a.lo = lo;
  a.hi = hi;
  a.runtime = runtime;
  a.key = "$" + name;
  return intern(std::move(a));
}

int ExprCtx::find_symbol(const std::string& name) const {
  auto it = index.find("$" + name);
  return it == index.end() ? -1 : it->second;
}

static void add_term(Expr& e, const Monomial& m, int64_t c) {
  if (!c) return;
  auto it = e.terms.find(m);
  if (it == e.terms.end()) {
    e.terms[m] = c;
  } else {
    it->second += c;
    if (!it->second) e.terms.erase(it);
  }
}

Expr operator+(const Expr& a, const Expr& b) {
  Expr r = a;
  for (auto& t : b.terms) add_term(r, t.first, t.second);
  return r;
}
Expr operator-(const Expr& a, const Expr& b) {
  Expr r = a;
  for (auto& t : b.terms) add_term(r, t.first, -t.second);
  return r;
}
static Monomial mono_mul(const Monomial& x, const Monomial& y) {
  Monomial r;
  size_t i = 0, j = 0;
  while (i < x.size() || j < y.size()) {
    if (j == y.size() || (i < x.size() && x[i].first < y[j].first)) r.push_back(x[i++]);
    else if (i == x.size() || y[j].first < x[i].first) r.push_back(y[j++]);
    else { r.push_back({x[i].first, x[i].second + y[j].second}); ++i; ++j; }
  }
  return r;
}
Expr operator*(const Expr& a, const Expr& b) {
  Expr r;
  for (auto& s : a.terms)
    for (auto& t : b.terms) add_term(r, mono_mul(s.first, t.first), s.second * t.second);
  return r;
}

// x / y for monomials; ok=false if y does not divide x.
static Monomial mono_div(const Monomial& x, const Monomial& y, bool* ok) {
  Monomial r;
  size_t j = 0;
  *ok = true;
  for (auto& p : x) {
    if (j < y.size() && y[j].first == p.first) {
      if (y[j].second > p.second) { *ok = false; return r; }
      if (p.second > y[j].second) r.push_back({p.first, p.second - y[j].second});
      ++j;
    } else {
      r.push_back(p);
    }
  }
  if (j != y.size()) *ok = false;
  return r;
}

Expr e_exact_div(const Expr& a, const Expr& b, bool* ok) {
  *ok = false;
  Expr r;
  if (b.terms.size() != 1) {
    if (a == b && !b.terms.empty()) { *ok = true; return Expr(1); }
    return r;
  }
  const Monomial& bm = b.terms.begin()->first;
  int64_t bc = b.terms.begin()->second;
  if (!bc) return r;
  for (auto& t : a.terms) {
    if (t.second % bc) return Expr();
    bool mok;
    Monomial m = mono_div(t.first, bm, &mok);
    if (!mok) return Expr();
    add_term(r, m, t.second / bc);
  }
  *ok = true;
  return r;
}

static int64_t fdiv(int64_t a, int64_t b) {
  int64_t q = a / b, r = a % b;
  return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q;
}

static Expr make_nl(ExprCtx& cx, AtomKind k, const char* nm, Expr a, Expr b) {
  Atom at;
  at.kind = k;
  at.key = std::string(nm) + "(" + e_str(cx, a) + "," + e_str(cx, b) + ")";
  at.a = std::make_shared<Expr>(std::move(a));
  at.b = std::make_shared<Expr>(std::move(b));
  return Expr::atom(cx.intern(std::move(at)));
}

Expr e_floordiv(ExprCtx& cx, const Expr& a, const Expr& b) {
  if (b.is_const()) {
    int64_t c = b.const_value();
    if (c == 1) return a;
    if (c > 0) {
      // floor((c*q + r) / c) = q + floor(r / c) for any integer-valued q
      Expr q, r;
      for (auto& t : a.terms) {
        int64_t qq = fdiv(t.second, c);
        add_term(q, t.first, qq);
        add_term(r, t.first, t.second - qq * c);
      }
      if (r.is_const()) return q + Expr(fdiv(r.const_value(), c));
      return q + make_nl(cx, AtomKind::FLOORDIV, "floordiv", r, b);
    }
  }
  bool ok;
  Expr q = e_exact_div(a, b, &ok);
  if (ok) return q;
  return make_nl(cx, AtomKind::FLOORDIV, "floordiv", a, b);
}

Expr e_ceildiv(ExprCtx& cx, const Expr& a, const Expr& b) { return e_floordiv(cx, a + b - Expr(1), b); }

Expr e_min(ExprCtx& cx, const Expr& a, const Expr& b) {
  if (a == b) return a;
  Expr d = a - b;
  if (d.is_const()) return d.const_value() < 0 ? a : b;
  if (e_str(cx, b) < e_str(cx, a)) return make_nl(cx, AtomKind::MIN, "min", b, a);
  return make_nl(cx, AtomKind::MIN, "min", a, b);
}
Expr e_max(ExprCtx& cx, const Expr& a, const Expr& b) {
  if (a == b) return a;
  Expr d = a - b;
  if (d.is_const()) return d.const_value() > 0 ? a : b;
  if (e_str(cx, b) < e_str(cx, a)) return make_nl(cx, AtomKind::MAX, "max", b, a);
  return make_nl(cx, AtomKind::MAX, "max", a, b);
}

std::string e_str(const ExprCtx& cx, const Expr& e) {
  if (e.terms.empty()) return "0";
  // order: higher-degree / named terms first, constant last, for readable canonical strings
  std::vector<std::pair<std::string, int64_t>> parts;
  int64_t cst = 0;
  for (auto& t : e.terms) {
    if (t.first.empty()) { cst = t.second; continue; }
    std::string m;
    for (auto& p : t.first) {
      const Atom& a = cx.atoms[p.first];
      std::string nm = a.kind == AtomKind::SYM ? a.name : a.key;
      for (int i = 0; i < p.second; ++i) { if (!m.empty()) m += "*"; m += nm; }
    }
    parts.push_back({m, t.second});
  }
  std::sort(parts.begin(), parts.end());
  std::ostringstream os;
  bool first = true;
  for (auto& p : parts) {
    int64_t c = p.second;
    if (first) { if (c == -1) os << "-"; else if (c != 1) os << c << "*"; }
    else { os << (c < 0 ? "-" : "+"); if (c != 1 && c != -1) os << (c < 0 ? -c : c) << "*"; }
    os << p.first;
    first = false;
  }
  if (cst || first) { if (!first && cst > 0) os << "+"; os << cst; }
  return os.str();
}

// mode 0: exact (every symbol must be bound); +1: upper bound; -1: lower bound. Unbound runtime
// symbols take their static bound; terms with a negative coefficient flip the mode.
static int64_t eval_rec(const ExprCtx& cx, const Expr& e, const std::vector<int64_t>& vals, bool* ok, int mode) {
  int64_t sum = 0;
  for (auto& t : e.terms) {
    int64_t prod = t.second;
    const int m = (t.second < 0) ? -mode : mode;
    for (auto& p : t.first) {
      const Atom& a = cx.atoms[p.first];
      int64_t v;
      if (a.kind == AtomKind::SYM) {
        v = p.first < static_cast<int>(vals.size()) ? vals[p.first] : INT64_MIN;
        if (v == INT64_MIN && m > 0) {
          if (a.hi_expr) v = eval_rec(cx, *a.hi_expr, vals, ok, 1);
          else if (a.hi != INT64_MAX) v = a.hi;
        } else if (v == INT64_MIN && m < 0) {
          v = a.lo;
        }
        if (v == INT64_MIN) { *ok = false; return 0; }
      } else {
        int64_t x = eval_rec(cx, *a.a, vals, ok, m);
        int64_t y = eval_rec(cx, *a.b, vals, ok, a.kind == AtomKind::FLOORDIV ? 0 : m);
        if (!*ok) return 0;
        if (a.kind == AtomKind::FLOORDIV) { if (y <= 0 && m != 0) { *ok = false; return 0; } if (y == 0) { *ok = false; return 0; } v = fdiv(x, y); }
        else if (a.kind == AtomKind::MIN) v = std::min(x, y);
        else v = std::max(x, y);
      }
      for (int i = 0; i < p.second; ++i) prod *= v;
    }
    sum += prod;
  }
  return sum;
}

int64_t e_eval(const ExprCtx& cx, const Expr& e, const std::vector<int64_t>& vals, bool* ok) {
  *ok = true;
  return eval_rec(cx, e, vals, ok, 0);
}
int64_t e_upper(const ExprCtx& cx, const Expr& e, const std::vector<int64_t>& vals, bool* ok) {
  *ok = true;
  return eval_rec(cx, e, vals, ok, 1);
}

int64_t e_eval_flat(const Expr& e, const std::vector<int64_t>& av, bool* ok) {
  *ok = true;
  int64_t sum = 0;
  for (auto& t : e.terms) {
    int64_t prod = t.second;
    for (auto& p : t.first) {
      const int64_t v = p.first < static_cast<int>(av.size()) ? av[p.first] : INT64_MIN;
      if (v == INT64_MIN) { *ok = false; return 0; }
      for (int i = 0; i < p.second; ++i) prod *= v;
    }
    sum += prod;
  }
  return sum;
}

void e_eval_atoms(const ExprCtx& cx, std::vector<int64_t>* vals) {
  vals->resize(cx.atoms.size(), INT64_MIN);
  for (size_t i = 0; i < cx.atoms.size(); ++i) {
    const Atom& a = cx.atoms[i];
    if (a.kind == AtomKind::SYM) continue;
    bool ok1, ok2;
    const int64_t x = e_eval_flat(*a.a, *vals, &ok1), y = e_eval_flat(*a.b, *vals, &ok2);
    if (!ok1 || !ok2 || (a.kind == AtomKind::FLOORDIV && y == 0)) { (*vals)[i] = INT64_MIN; continue; }
    (*vals)[i] = a.kind == AtomKind::FLOORDIV ? fdiv(x, y) : a.kind == AtomKind::MIN ? std::min(x, y) : std::max(x, y);
  }
}

bool e_has_runtime(const ExprCtx& cx, const Expr& e) {
  for (auto& t : e.terms)
    for (auto& p : t.first) {
      const Atom& a = cx.atoms[p.first];
      if (a.kind == AtomKind::SYM) { if (a.runtime) return true; }
      else if (e_has_runtime(cx, *a.a) || e_has_runtime(cx, *a.b)) return true;
    }
  return false;
}

}  // namespace sod2
