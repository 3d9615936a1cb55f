// Per-request binding (evaluate every RDP expression), view resolution, liveness and the
// run-time memory allocation plan (Section 4.4.1: one linear arena, planned at execution time once
// all sizes are known, greedy from the peak-memory step outwards).
#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>

#include "engine.h"

namespace sod2 {

// ---- recycled host blocks for the per-batch tables (engine.h)
namespace {
struct BlockPool {
  std::mutex mu;
  std::vector<std::pair<unsigned char*, size_t>> free_blocks;   // at most POOL_MAX, each at most BLOCK_MAX bytes
};
constexpr size_t POOL_MAX = 8, BLOCK_MAX = size_t(16) << 20;   // at most 128 MB parked
// never destroyed: handles may be released after the static destructors of this library have run
BlockPool& block_pool() { static BlockPool* p = new BlockPool; return *p; }
}  // namespace

unsigned char* block_acquire(size_t need, size_t* cap) {
  BlockPool& P = block_pool();
  {
    std::lock_guard<std::mutex> lk(P.mu);
    // the smallest recycled block that fits
    int best = -1;
    for (size_t i = 0; i < P.free_blocks.size(); ++i)
      if (P.free_blocks[i].second >= need && (best < 0 || P.free_blocks[i].second < P.free_blocks[best].second)) best = static_cast<int>(i);
    if (best >= 0) {
      auto b = P.free_blocks[best];
      P.free_blocks.erase(P.free_blocks.begin() + best);
      *cap = b.second;
      return b.first;
    }
  }
  *cap = need;
  return new unsigned char[need];
}

void block_release(unsigned char* p, size_t cap) {
  BlockPool& P = block_pool();
  if (cap <= BLOCK_MAX) {
    std::lock_guard<std::mutex> lk(P.mu);
    if (P.free_blocks.size() < POOL_MAX) { P.free_blocks.push_back({p, cap}); return; }
  }
  delete[] p;
}

Status bind_dims(const Compiled* c, int n_req, int n_syms, const char* const* names, const int64_t* values, Binding* out) {
  const Graph& g = c->g;
  if (n_req <= 0 || n_syms < 0) { out->err = "need at least one request"; return E_INVALID_ARG; }
  out->c = c;
  out->n_req = n_req;
  out->vals.assign(n_req, std::vector<int64_t>(g.cx.atoms.size(), INT64_MIN));
  for (int s = 0; s < n_syms; ++s) {
    int id = g.cx.find_symbol(names[s]);
    if (id < 0) { out->err = std::string("unknown symbol ") + names[s]; return E_INVALID_ARG; }
    const Atom& a = g.cx.atoms[id];
    for (int r = 0; r < n_req; ++r) {
      int64_t v = values[static_cast<size_t>(r) * n_syms + s];
      if (v < a.lo || v > a.hi) { out->err = "symbol " + a.name + " = " + std::to_string(v) + " outside its declared range"; return E_BAD_DIM; }
      out->vals[r][id] = v;
    }
  }
  for (int id : g.user_syms)
    if (out->vals[0][id] == INT64_MIN) { out->err = "symbol " + g.cx.atoms[id].name + " is not bound"; return E_UNBOUND_SYMBOL; }
  static const bool prof = getenv("SOD2_HOST_PROFILE") != nullptr;
  auto t0 = std::chrono::steady_clock::now();
  // bind-time assertions recorded by RDP (two inferences of one extent must agree)
  for (int r = 0; r < n_req; ++r)
    for (auto& as : g.asserts) {
      bool ok1, ok2;
      int64_t x = e_eval(g.cx, as.a, out->vals[r], &ok1), y = e_eval(g.cx, as.b, out->vals[r], &ok2);
      if (ok1 && ok2 && x != y && !(as.kind == 1 && (x == 1 || y == 1))) {
        out->err = "shape conflict: " + as.what + " (" + std::to_string(x) + " vs " + std::to_string(y) + ")";
        return E_SHAPE_CONFLICT;
      }
    }
  auto t1 = std::chrono::steady_clock::now();
  Status es = evaluate_dims(out);
  if (es != OK) return es;
  if (prof) {
    auto t3 = std::chrono::steady_clock::now();
    auto us = [](auto a, auto b) { return std::chrono::duration<double, std::micro>(b - a).count(); };
    fprintf(stderr, "[sod2] bind: %zu assertions %.1f us, %zu extent expressions and %zu tensors %.1f us\n", g.asserts.size(), us(t0, t1),
            c->dim_exprs.size(), g.tensors.size(), us(t1, t3));
  }
  return OK;
}

// Extents of every tensor for every request from the bound symbol values (out->vals): all non-linear atoms once per
// request (children first), then every distinct extent expression once per request as a flat polynomial; tensors
// pick their extents from that table.  An extent that depends on an unbound run-time symbol takes its static
// upper bound.
Status evaluate_dims(Binding* out) {
  const Compiled* c = out->c;
  const Graph& g = c->g;
  const int n_req = out->n_req;
  const size_t U = c->dim_exprs.size();
  std::vector<int64_t> uval(static_cast<size_t>(n_req) * U);
  std::vector<char> uok(static_cast<size_t>(n_req) * U);
  std::vector<int64_t> atom_vals;
  for (int r = 0; r < n_req; ++r) {
    atom_vals = out->vals[r];
    e_eval_atoms(g.cx, &atom_vals);
    for (size_t u = 0; u < U; ++u) {
      bool ok;
      int64_t v = e_eval_flat(c->dim_exprs[u], atom_vals, &ok);
      if (!ok) v = e_upper(g.cx, c->dim_exprs[u], out->vals[r], &ok);   // depends on a runtime symbol: static upper bound for planning
      uval[r * U + u] = v;
      uok[r * U + u] = ok;
    }
  }
  // extents equal for every request of this batch: their tensors get one shared table entry
  std::vector<char> usame(U, 1);
  for (size_t u = 0; u < U; ++u)
    for (int r = 1; r < n_req; ++r)
      if (uval[r * U + u] != uval[u] || uok[r * U + u] != uok[u]) { usame[u] = 0; break; }
  out->dims.reset(g.tensors.size(), n_req);
  std::vector<int> class_rep(c->n_dim_classes, -1);   // the tensor whose row the class's other members read
  for (size_t t = 0; t < g.tensors.size(); ++t) {
    const ShapeVal& s = g.tensors[t].S;
    if (s.rank < 0) continue;
    const int dc = t < c->dim_class.size() ? c->dim_class[t] : -1;
    if (dc >= 0 && class_rep[dc] >= 0) { out->dims.alias(t, class_rep[dc]); continue; }
    if (dc >= 0) class_rep[dc] = static_cast<int>(t);
    if (s.rank > MAX_RANK) { out->err = "rank above " + std::to_string(MAX_RANK) + " for " + g.tensors[t].name; return E_UNSUPPORTED_OP; }
    const std::vector<int>& ids = c->dim_expr_id[t];
    bool evaluable = true;
    for (int i = 0; i < s.rank; ++i) if (ids[i] < 0) evaluable = false;
    for (int r = 0; r < n_req && evaluable; ++r)
      for (int i = 0; i < s.rank; ++i) if (!uok[r * U + ids[i]]) { evaluable = false; break; }
    if (!evaluable) continue;
    bool same = true;
    for (int i = 0; i < s.rank; ++i) if (!usame[ids[i]]) same = false;
    auto per = same ? out->dims.make_shared(t) : out->dims.make(t);
    for (int r = 0; r < (same ? 1 : n_req); ++r) {
      per[r].n = s.rank;
      for (int i = 0; i < s.rank; ++i) {
        const int64_t v = uval[r * U + ids[i]];
        if (v < 0) { out->err = "negative extent for " + g.tensors[t].name; return E_BAD_DIM; }
        per[r].v[i] = v;
      }
    }
  }
  return OK;
}

// A binding with some run-time symbols bound to the counts their operators produced (exact handling of
// execution-determined extents): the same user symbols, `rt_vals[r]` = (atom, value) pairs for request r.
Status rebind_runtime(const Binding& base, const std::vector<std::vector<std::pair<int, int64_t>>>& rt_vals, Binding* out) {
  out->c = base.c;
  out->n_req = base.n_req;
  out->vals = base.vals;
  for (int r = 0; r < base.n_req && r < static_cast<int>(rt_vals.size()); ++r)
    for (auto& av : rt_vals[r]) {
      if (av.first < 0 || av.first >= static_cast<int>(out->vals[r].size()) || av.second < 0) { out->err = "bad run-time symbol value"; return E_BAD_DIM; }
      out->vals[r][av.first] = av.second;
    }
  return evaluate_dims(out);
}

namespace {

int64_t numel(const DimVec& d) {
  int64_t n = 1;
  for (int64_t v : d) n *= v;
  return n;
}
DimVec contiguous_strides(const DimVec& d) {
  DimVec s(d.size(), 0);
  int64_t acc = 1;
  for (int i = static_cast<int>(d.size()) - 1; i >= 0; --i) { s[i] = acc; acc *= d[i]; }
  return s;
}

// strides of `newd` viewing memory laid out as (oldd, olds); false if a copy would be needed
bool reshape_view(const DimVec& oldd, const DimVec& olds, const DimVec& newd, DimVec* news) {
  news->assign(newd.size(), 0);
  if (numel(oldd) == 0) { *news = contiguous_strides(newd); return true; }
  int vd = static_cast<int>(newd.size()) - 1;
  if (oldd.empty()) { for (auto& s : *news) s = 1; return true; }
  int64_t chunk_base = olds.back(), tnumel = 1, vnumel = 1;
  for (int td = static_cast<int>(oldd.size()) - 1; td >= 0; --td) {
    tnumel *= oldd[td];
    if (td == 0 || (oldd[td - 1] != 1 && olds[td - 1] != tnumel * chunk_base)) {
      while (vd >= 0 && (vnumel < tnumel || newd[vd] == 1)) {
        (*news)[vd] = vnumel * chunk_base;
        vnumel *= newd[vd];
        --vd;
      }
      if (vnumel != tnumel) return false;
      if (td > 0) { chunk_base = olds[td - 1]; tnumel = 1; vnumel = 1; }
    }
  }
  return vd == -1;
}

struct Planner {
  const Compiled& c;
  const Graph& g;
  const Binding& b;
  Plan& p;
  std::vector<char> resolved;
  std::vector<int> class_rep;    // per view class: the first tensor resolved in this plan, whose rows the others read
  Planner(const Compiled& cc, const Binding& bb, Plan& pp)
      : c(cc), g(cc.g), b(bb), p(pp), resolved(cc.g.tensors.size(), 0), class_rep(cc.n_view_classes, -1) {}

  Status fail(Status s, const std::string& m) { p.err = m; return s; }

  Status make_root(int t) {
    if (b.dims[t].empty()) return fail(E_INTERNAL, "no concrete shape for " + g.tensors[t].name);
    const Tensor& T = g.tensors[t];
    RootBuf& R = p.roots[t];
    p.root_of[t] = t;
    const int vc = c.view_class[t];
    if (vc >= 0 && class_rep[vc] >= 0) {
      // same extents, element size and layout rule as a root already made: read its rows
      const int rep = class_rep[vc];
      p.views.alias(t, rep);
      p.inst_off.alias(t, rep);
      const RootBuf& Q = p.roots[rep];
      R.bytes = Q.bytes;
      R.stats_off = Q.stats_off;
      R.stats_rows = Q.stats_rows;
      R.stats_slots = Q.stats_slots;
      set_where(T, &R);
      resolved[t] = 1;
      return OK;
    }
    if (vc >= 0) class_rep[vc] = t;
    auto inst_off = p.inst_off.make(t);
    int64_t off = 0;
    int esz = dtype_size(T.dtype);
    bool per_request = T.kind != TKind::CONST;
    const int nv = open_views(t, -1);
    auto views = p.views[t];
    auto dims = b.dims[t];
    for (int r = 0; r < nv; ++r) {
      View& v = views[r];
      v.offset = 0;
      v.dims = dims[r];
      v.strides = contiguous_strides(v.dims);
      // convolution graphs keep rank-4 float intermediates channels-last: [N,C,H,W] with C innermost
      if (g.has_conv && v.dims.size() == 4 && T.kind == TKind::VALUE && !T.is_output &&
          (T.dtype == DType::BF16 || T.dtype == DType::F32)) {
        const int64_t C = v.dims[1], H = v.dims[2], W = v.dims[3];
        v.strides = {H * W * C, 1, W * C, C};
      }
    }
    for (int r = 0; r < p.n_req; ++r) {
      inst_off[r] = per_request ? off : 0;
      int64_t bytes = numel(dims[r]) * esz;
      if (per_request) off += (bytes + 15) & ~int64_t(15);
      else off = bytes;
    }
    if (t < static_cast<int>(c.stats_width.size()) && c.stats_width[t] > 0) {
      // LayerNorm row statistics written by the producing GEMM live behind the tensor's instances: one
      // (mean, M2) float pair per packed row and slot of 32 columns (the most any tile version writes)
      const int64_t row_bytes = static_cast<int64_t>(c.stats_width[t]) * esz;
      if (!per_request || off % row_bytes) return fail(E_INTERNAL, "row statistics need densely packed rows: " + T.name);
      R.stats_rows = off / row_bytes;
      R.stats_slots = c.stats_width[t] / 32;
      R.stats_off = off;
      off += R.stats_rows * R.stats_slots * 8;
    }
    R.bytes = off;
    set_where(T, &R);
    resolved[t] = 1;
    return OK;
  }
  static void set_where(const Tensor& T, RootBuf* R) {
    if (T.kind == TKind::INPUT) { R->where = RootBuf::INPUT; R->io_index = T.io_index; }
    else if (T.kind == TKind::CONST) { R->where = RootBuf::CONST; }
    else if (T.is_output) { R->where = RootBuf::OUTPUT; R->io_index = T.io_index; }
    else R->where = RootBuf::ARENA;
  }

  // Views of `t`: one entry per request, or one shared entry when neither its extents nor the views it derives from
  // (`other`, if any) depend on the request.  Returns the number of entries to fill.
  int open_views(int t, int other) {
    const bool same = b.dims.shared(t) && (other < 0 || p.views.shared(other));
    if (same) p.views.make_shared(t); else p.views.make(t);
    return same ? 1 : p.n_req;
  }

  Status resolve(int t) {
    if (resolved[t]) return OK;
    const Storage& st = c.storage[t];
    if (st.kind == Storage::FOLDED) { resolved[t] = 1; return OK; }
    if (st.kind == Storage::ROOT) return make_root(t);
    if (b.dims[t].empty()) return fail(E_INTERNAL, "no concrete shape for " + g.tensors[t].name);
    {
      // a view of the same class as one already resolved: same rows, the bytes belong to this one's own source
      const int vc = c.view_class[t];
      if (vc >= 0 && st.other >= 0) {
        Status s = resolve(st.other);
        if (s != OK) return s;
        if (class_rep[vc] >= 0) {
          p.views.alias(t, class_rep[vc]);
          p.root_of[t] = p.root_of[st.other];
          resolved[t] = 1;
          return OK;
        }
        class_rep[vc] = t;
      }
      if (st.other >= 0) {
        Status s = resolve(st.other);
        if (s != OK) return s;
        p.root_of[t] = p.root_of[st.other];
      }
    }
    if (st.kind == Storage::ALIAS) {
      Status s = resolve(st.other);
      if (s != OK) return s;
      const int nv = open_views(t, st.other);
      for (int r = 0; r < nv; ++r) {
        const View& vo = p.views[st.other][r];
        View& v = p.views[t][r];
        v.offset = vo.offset;
        v.dims = b.dims[t][r];
        v.strides = vo.strides;
        if (v.dims != vo.dims) return fail(E_INTERNAL, "aliased tensors differ in shape: " + g.tensors[t].name);
      }
      resolved[t] = 1;
      return OK;
    }
    if (st.kind == Storage::INDIRECT_IN || st.kind == Storage::INDIRECT_OUT) {
      // the samples of `other` selected by an id list: same storage, same strides, own (upper-bound) extents
      Status s = resolve(st.other);
      if (s != OK) return s;
      const int nv = open_views(t, st.other);
      for (int r = 0; r < nv; ++r) {
        const View& vo = p.views[st.other][r];
        View& v = p.views[t][r];
        v.offset = vo.offset;
        v.dims = b.dims[t][r];
        v.strides = vo.strides;
        v.ind_gate = st.gate;
        v.ind_list = st.list;
      }
      resolved[t] = 1;
      return OK;
    }
    if (st.kind == Storage::VIEW_OF_OUTPUT) {
      // t is the input of a Transpose whose output `o` owns the bytes
      int o = st.other;
      Status s = resolve(o);
      if (s != OK) return s;
      const std::vector<int64_t>& perm = c.view_param[t].a;
      const int nv = open_views(t, o);
      for (int r = 0; r < nv; ++r) {
        const View& vo = p.views[o][r];
        View& v = p.views[t][r];
        v.offset = vo.offset;
        v.dims = b.dims[t][r];
        v.strides.assign(v.dims.size(), 0);
        for (size_t i = 0; i < perm.size(); ++i) v.strides[perm[i]] = vo.strides[i];
      }
      resolved[t] = 1;
      return OK;
    }
    // VIEW_OF_INPUT
    int in = st.other;
    Status s = resolve(in);
    if (s != OK) return s;
    const Compiled::ViewParam& vp = c.view_param[t];
    const int kind = vp.op;
    const std::vector<int64_t>& perm = vp.a;
    const std::vector<int64_t>& sl_start = vp.a;
    const std::vector<int64_t>& sl_step = vp.b;
    if (kind == 2 && sl_start.size() != p.views[in][0].dims.size()) return fail(E_INTERNAL, "slice parameters of " + g.tensors[t].name);
    const int nv = open_views(t, in);
    for (int r = 0; r < nv; ++r) {
      const View& vi = p.views[in][r];
      View& v = p.views[t][r];
      v.offset = vi.offset;
      v.dims = b.dims[t][r];
      if (kind == 0) {
        v.strides.resize(perm.size());
        for (size_t i = 0; i < perm.size(); ++i) v.strides[i] = vi.strides[perm[i]];
      } else if (kind == 1) {
        if (!reshape_view(vi.dims, vi.strides, v.dims, &v.strides))
          return fail(E_UNSUPPORTED_OP, "Reshape producing " + g.tensors[t].name + " is not a view of its input layout");
      } else {  // Slice
        v.strides = vi.strides;
        for (size_t ax = 0; ax < vi.dims.size(); ++ax) {
          const int64_t st0 = sl_start[ax], step = sl_step[ax];
          v.offset += st0 * vi.strides[ax];
          v.strides[ax] = vi.strides[ax] * step;
        }
      }
    }
    resolved[t] = 1;
    return OK;
  }

  Status run() {
    auto t0 = std::chrono::steady_clock::now();
    size_t T = g.tensors.size();
    p.inst_off.reset(T, p.n_req);
    p.views.reset(T, p.n_req);   // rows are made per tensor when it is resolved
    p.root_of.assign(T, -1);
    p.roots.assign(T, RootBuf());
    // resolve every tensor a group touches
    for (auto& G : c.groups) {
      if (G.kind == GKind::UNSUPPORTED) return fail(E_UNSUPPORTED_OP, "group around " + g.nodes[G.nodes[0]].op + ": " + G.why);
      for (int t : G.ext_in) { Status s = resolve(t); if (s != OK) return s; }
      for (int t : G.ext_out) { Status s = resolve(t); if (s != OK) return s; }
    }
    for (int t : g.outputs) { Status s = resolve(t); if (s != OK) return s; }
    // an input of which only the shape is read still has an instance per request in the caller's buffer
    for (int t : g.inputs) if (!b.dims[t].empty()) { Status s = resolve(t); if (s != OK) return s; }
    static const bool prof = getenv("SOD2_HOST_PROFILE") != nullptr;
    auto t1 = std::chrono::steady_clock::now();
    // GEMM groups that will run as one persistent kernel: their members overlap in time
    {
      Status cs = detect_chains(&p);
      if (cs != OK) return cs;
    }
    // liveness of arena roots over the group sequence
    int steps = static_cast<int>(c.groups.size());
    for (int s = 0; s < steps; ++s) {
      const Group& G = c.groups[s];
      // a member of a chain reads and writes at any time between the chain's first and last step
      int lo = s, hi = s;
      if (s < static_cast<int>(p.chain_of.size()) && p.chain_of[s] >= 0) {
        const Plan::Chain& ch = p.chains[p.chain_of[s]];
        lo = ch.groups.front();
        hi = ch.groups.back();
      }
      auto touch = [&](int t, bool def) {
        if (c.storage[t].kind == Storage::FOLDED || !resolved[t]) return;
        int root = p.root_of[t];
        if (root < 0) return;
        RootBuf& R = p.roots[root];
        if (R.def_step < 0 || lo < R.def_step) R.def_step = lo;
        R.last_step = std::max(R.last_step, hi);
        (void)def;
      };
      for (int t : G.ext_out) touch(t, true);
      for (int t : G.ext_in) touch(t, false);
    }
    auto t2 = std::chrono::steady_clock::now();
    Status s = plan_arena(steps);
    if (prof) {
      auto t3 = std::chrono::steady_clock::now();
      auto us = [](auto a, auto b) { return std::chrono::duration<double, std::micro>(b - a).count(); };
      int n_res = 0, n_rep = 0;
      for (size_t t = 0; t < T; ++t) n_res += resolved[t] && c.storage[t].kind != Storage::FOLDED;
      for (int r : class_rep) n_rep += r >= 0;
      fprintf(stderr, "[sod2] plan: views %.1f us (%d tensors, %d table rows filled), liveness %.1f us, arena %.1f us\n", us(t0, t1), n_res, n_rep, us(t1, t2), us(t2, t3));
    }
    return s;
  }

  // Peak-first greedy: place the tensors live at the peak step contiguously, then walk forward
  // and backward from the peak, each new tensor taking the smallest free gap that fits (ties: lowest
  // offset), else extending the arena. Offsets are 256-byte aligned; the first 256 bytes hold the
  // device status word.
  Status plan_arena(int steps) {
    // header: status word (256 B) + one 8-byte count slot per (runtime symbol, request)
    // ... + the row-block counters of the GEMM chains
    p.chain_counter_off = (256 + 8 * g.cx.atoms.size() * static_cast<size_t>(p.n_req) + 15) & ~size_t(15);
    const size_t HEADER0 = (p.chain_counter_off + 4 * p.chain_counter_words + 255) & ~size_t(255);
    p.header_clear_bytes = p.chain_counter_words ? HEADER0 : 256;
    // staged (exact) plans keep the group scratch and the Switch index lists at fixed places right behind the
    // header, so that they do not move when a later stage plans the tensors again
    p.header_end = HEADER0;
    const size_t HEADER = HEADER0 + p.front_reserve;
    std::vector<int> ids;
    for (size_t t = 0; t < p.roots.size(); ++t)
      if (p.roots[t].where == RootBuf::ARENA && p.roots[t].def_step >= 0 && p.roots[t].def_step <= p.place_until_step &&
          p.roots[t].last_step >= p.place_from_step)
        ids.push_back(static_cast<int>(t));
    const size_t band = (c.flags & OPT_GUARD_BANDS) ? 256 : 0;
    auto sz = [&](int t) { return ((static_cast<size_t>(p.roots[t].bytes) + 255) & ~size_t(255)) + band; };
    // scratch of groups is planned like a tensor living for exactly that step
    std::vector<size_t> live(steps + 1, 0);
    p.sum_bytes = 0;
    for (int t : ids) {
      p.sum_bytes += sz(t);
      for (int s = p.roots[t].def_step; s <= p.roots[t].last_step; ++s) live[s] += sz(t);
    }
    int peak = 0;
    for (int s = 0; s < steps; ++s) if (live[s] > live[peak]) peak = s;
    p.peak_step = peak;
    p.peak_live_bytes = steps ? live[peak] : 0;
    struct Placed { size_t off, size; int def, last; };
    std::vector<Placed> placed;
    size_t top = HEADER;
    // smallest_gap: the smallest free gap that fits (ties: lowest offset); otherwise the lowest one
    auto place = [&](int t, bool smallest_gap) {
      RootBuf& R = p.roots[t];
      size_t need = sz(t);
      // guard bands only mean something where no other tensor ever covers them: every tensor its own slot
      if (c.flags & (OPT_NO_REUSE | OPT_GUARD_BANDS)) { R.arena_off = top; top += need; placed.push_back({R.arena_off, need, R.def_step, R.last_step}); return; }
      // free gaps among tensors whose lifetime overlaps this one
      std::vector<std::pair<size_t, size_t>> busy;
      for (auto& q : placed) if (!(q.last < R.def_step || q.def > R.last_step)) busy.push_back({q.off, q.off + q.size});
      std::sort(busy.begin(), busy.end());
      size_t best_off = SIZE_MAX, best_gap = SIZE_MAX, cur = HEADER;
      for (auto& iv : busy) {
        if (iv.first > cur && iv.first - cur >= need && iv.first - cur < best_gap) {
          best_gap = iv.first - cur;
          best_off = cur;
          if (!smallest_gap) break;
        }
        cur = std::max(cur, iv.second);
      }
      if (best_off == SIZE_MAX) best_off = cur;  // after the last overlapping tensor (may extend the arena)
      R.arena_off = best_off;
      top = std::max(top, best_off + need);
      placed.push_back({best_off, need, R.def_step, R.last_step});
    };
    std::vector<char> done(p.roots.size(), 0);
    // 0. tensors an earlier stage has already placed (and filled) stay where they are
    for (auto& pin : p.pinned) {
      const int t = pin.first;
      if (t < 0 || t >= static_cast<int>(p.roots.size()) || p.roots[t].where != RootBuf::ARENA || p.roots[t].def_step < 0) continue;
      if (std::find(ids.begin(), ids.end(), t) == ids.end()) continue;
      if (pin.second < HEADER) return fail(E_INTERNAL, "pinned tensor inside the arena header");
      p.roots[t].arena_off = pin.second;
      placed.push_back({pin.second, sz(t), p.roots[t].def_step, p.roots[t].last_step});
      top = std::max(top, pin.second + sz(t));
      done[t] = 1;
    }
    // 1. live set at the peak, in (def step, id) order
    std::vector<int> at_peak;
    for (int t : ids) if (!done[t] && p.roots[t].def_step <= peak && p.roots[t].last_step >= peak) at_peak.push_back(t);
    std::sort(at_peak.begin(), at_peak.end(), [&](int x, int y) { return std::make_pair(p.roots[x].def_step, x) < std::make_pair(p.roots[y].def_step, y); });
    for (int t : at_peak) { place(t, true); done[t] = 1; }
    // 2. forward from the peak
    std::vector<int> fwd;
    for (int t : ids) if (!done[t] && p.roots[t].def_step > peak) fwd.push_back(t);
    std::sort(fwd.begin(), fwd.end(), [&](int x, int y) { return std::make_pair(p.roots[x].def_step, x) < std::make_pair(p.roots[y].def_step, y); });
    for (int t : fwd) { place(t, true); done[t] = 1; }
    // 3. backward from the peak: tensors dead before it, latest last-use first
    std::vector<int> bwd;
    for (int t : ids) if (!done[t]) bwd.push_back(t);
    std::sort(bwd.begin(), bwd.end(), [&](int x, int y) { return std::make_pair(-p.roots[x].last_step, x) < std::make_pair(-p.roots[y].last_step, y); });
    for (int t : bwd) { place(t, true); done[t] = 1; }
    // 4. where memory does not fall off monotonically on both sides of the peak (branches whose small
    // results outlive their large intermediates), the walk above fragments.  If it ended more than 2 %
    // above the live peak, a second placement is tried, largest tensor first at the lowest offset
    // that is free over its lifetime, and the smaller arena is kept.
    if (p.pinned.empty() && !(c.flags & (OPT_NO_REUSE | OPT_GUARD_BANDS)) && top - HEADER > p.peak_live_bytes + p.peak_live_bytes / 50) {
      std::vector<size_t> first_off(ids.size());
      for (size_t i = 0; i < ids.size(); ++i) first_off[i] = p.roots[ids[i]].arena_off;
      const size_t first_top = top;
      placed.clear();
      top = HEADER;
      std::vector<int> by_size = ids;
      std::sort(by_size.begin(), by_size.end(), [&](int x, int y) {
        return std::make_tuple(~sz(x), p.roots[x].def_step, x) < std::make_tuple(~sz(y), p.roots[y].def_step, y);
      });
      for (int t : by_size) place(t, false);
      if (top >= first_top) {
        for (size_t i = 0; i < ids.size(); ++i) p.roots[ids[i]].arena_off = first_off[i];
        top = first_top;
      }
    }
    p.arena_bytes = top;
    p.guard_bands.clear();
    if (band)
      for (int t : ids) p.guard_bands.push_back({p.roots[t].arena_off + sz(t) - band, t});
    return OK;
  }
};

}  // namespace

Status make_plan(const Compiled* c, const Binding* b, Plan* p) {
  p->c = c;
  p->b = b;
  p->n_req = b->n_req;
  static const bool prof = getenv("SOD2_HOST_PROFILE") != nullptr;
  auto t0 = std::chrono::steady_clock::now();
  Planner pl(*c, *b, *p);
  Status s = pl.run();
  if (s != OK) return s;
  auto t1 = std::chrono::steady_clock::now();
  s = build_launches(p);
  if (prof) {
    auto t2 = std::chrono::steady_clock::now();
    fprintf(stderr, "[sod2] plan: views+liveness+arena %.1f us, launches %.1f us\n", std::chrono::duration<double, std::micro>(t1 - t0).count(),
            std::chrono::duration<double, std::micro>(t2 - t1).count());
  }
  return s;
}

}  // namespace sod2
