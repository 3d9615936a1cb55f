// Static execution planning (Section 4.3 of the paper).
//
// A DAG of fused groups admits several execution orders and the order decides how many bytes of
// intermediate results are live at once.  Finding the best order of a whole model is NP-complete,
// so the paper partitions the graph at operators whose output shape is nac and treats each
// sub-graph on its own: with known-constant shapes an exhaustive search gives the optimum; with
// symbolic or operation-inferred shapes the memory requirements of two orders can still be
// compared, most reliably when they derive from the same symbols.
//
// Here: the sub-graphs are those of the nac partition (fuse.cpp), run in index order.  Inside a
// sub-graph every topological order is covered by a search over the sets of groups already run: the
// live bytes after a set do not depend on the order inside it, so the best peak of a set is the
// minimum over its last group, and only down-closed sets are reachable.  Tensor sizes are the RDP
// extent expressions evaluated at two corners of the declared symbol ranges: every symbol at its
// upper bound (the primary objective, exact) and at its lower bound (tie-break); an
// execution-determined extent counts with its static upper bound, which is what the run-time
// arena reserves for it.  A search that outgrows its state budget, or a size that cannot be
// bounded, leaves that sub-graph in its default order.  The default order is also kept whenever the
// search does not find a strictly smaller peak, so chains (all benchmark models) are untouched.
#include <algorithm>
#include <cstring>
#include <string>
#include <unordered_map>

#include "engine.h"

namespace sod2 {
namespace {

constexpr int64_t UNDECLARED_HI = 1024;   // stand-in upper corner for a symbol declared without a range
constexpr size_t STATE_BUDGET = 200000;   // sets of finished groups kept per sub-graph
constexpr int MAX_SG_GROUPS = 512;

struct Root {
  std::vector<int> touch;   // groups reading or writing the storage (creation indices), unique
  int64_t bytes[2] = {0, 0};
};

int root_of(const Compiled& c, int t) {
  for (int hop = 0; hop < 64 && t >= 0; ++hop) {
    const Storage& s = c.storage[t];
    if (s.kind == Storage::ROOT) return t;
    if (s.kind == Storage::FOLDED) return -1;
    t = s.other;
  }
  return -1;
}

using Mask = std::vector<uint64_t>;
inline bool mtest(const Mask& m, int i) { return (m[i >> 6] >> (i & 63)) & 1; }
inline void mset(Mask& m, int i) { m[i >> 6] |= uint64_t(1) << (i & 63); }
inline std::string mkey(const Mask& m) { return std::string(reinterpret_cast<const char*>(m.data()), m.size() * 8); }

struct Entry {
  Mask mask;
  int64_t peak[2], live[2];
  int parent, last;
};

// lexicographic comparison of (upper corner, lower corner)
inline bool better(const int64_t a[2], const int64_t b[2]) { return a[0] != b[0] ? a[0] < b[0] : a[1] < b[1]; }

// peak of live bytes of a complete order, both corners
void simulate(const std::vector<Root>& roots, const std::vector<int>& order, int64_t peak[2]) {
  const size_t G = order.size();
  std::vector<int> pos(G);
  for (size_t i = 0; i < G; ++i) pos[order[i]] = static_cast<int>(i);
  for (int k = 0; k < 2; ++k) {
    std::vector<int64_t> diff(G + 1, 0);
    for (const Root& r : roots) {
      if (r.touch.empty()) continue;
      int first = static_cast<int>(G), last = -1;
      for (int g : r.touch) { first = std::min(first, pos[g]); last = std::max(last, pos[g]); }
      diff[first] += r.bytes[k];
      diff[last + 1] -= r.bytes[k];
    }
    int64_t live = 0;
    peak[k] = 0;
    for (size_t i = 0; i < G; ++i) { live += diff[i]; peak[k] = std::max(peak[k], live); }
  }
}

}  // namespace

// deps[g]: groups that must run before g.  `order` holds the default order on entry and the planned
// order on return.  Indices are positions in c->groups.
void plan_execution_order(Compiled* c, const std::vector<std::vector<int>>& deps, std::vector<int>* order) {
  const Graph& g = c->g;
  const int G = static_cast<int>(c->groups.size());
  OrderStats& st = c->order_stats;
  st = OrderStats();
  if (G == 0) return;

  // sizes of the arena tensors at the two corners
  std::vector<int64_t> corner[2];
  for (int k = 0; k < 2; ++k) {
    corner[k].assign(g.cx.atoms.size(), INT64_MIN);
    for (int id : g.user_syms) {
      const Atom& a = g.cx.atoms[id];
      corner[k][id] = k == 0 ? (a.hi != INT64_MAX ? a.hi : std::max<int64_t>(a.lo, UNDECLARED_HI)) : a.lo;
    }
  }
  std::vector<int> root_index(g.tensors.size(), -1);
  std::vector<Root> roots;
  bool sizes_ok = true;
  auto touch = [&](int t, int gi) {
    const int r = root_of(*c, t);
    if (r < 0) return;
    const Tensor& T = g.tensors[r];
    if (T.kind != TKind::VALUE || T.is_output) return;   // inputs, weights and outputs are the caller's memory
    if (root_index[r] < 0) {
      root_index[r] = static_cast<int>(roots.size());
      roots.emplace_back();
      Root& R = roots.back();
      for (int k = 0; k < 2; ++k) {
        int64_t n = dtype_size(T.dtype);
        if (T.S.rank < 0) sizes_ok = false;
        for (int i = 0; i < T.S.rank && sizes_ok; ++i) {
          if (!T.S.dims[i].known()) { sizes_ok = false; break; }
          bool ok;
          const int64_t v = e_upper(g.cx, T.S.dims[i].e, corner[k], &ok);
          if (!ok || v < 0) { sizes_ok = false; break; }
          n *= v;
        }
        R.bytes[k] = (n + 255) & ~int64_t(255);
      }
    }
    Root& R = roots[root_index[r]];
    if (std::find(R.touch.begin(), R.touch.end(), gi) == R.touch.end()) R.touch.push_back(gi);
  };
  for (int gi = 0; gi < G; ++gi) {
    for (int t : c->groups[gi].ext_out) touch(t, gi);
    for (int t : c->groups[gi].ext_in) touch(t, gi);
  }
  if (!sizes_ok) { st.unbounded = 1; return; }
  simulate(roots, *order, st.default_peak);
  st.planned_peak[0] = st.default_peak[0];
  st.planned_peak[1] = st.default_peak[1];

  // groups of each sub-graph, in default order
  int n_sub = 0;
  for (const Group& G2 : c->groups) n_sub = std::max(n_sub, G2.subgraph + 1);
  std::vector<std::vector<int>> members(n_sub);
  for (int gi : *order) members[c->groups[gi].subgraph].push_back(gi);
  std::vector<int> planned;
  planned.reserve(G);
  bool any_change = false;

  for (int sg = 0; sg < n_sub; ++sg) {
    const std::vector<int>& M = members[sg];
    const int n = static_cast<int>(M.size());
    auto keep_default = [&]() { planned.insert(planned.end(), M.begin(), M.end()); };
    if (n <= 2) { keep_default(); continue; }
    if (n > MAX_SG_GROUPS) { ++st.abandoned_subgraphs; keep_default(); continue; }
    std::vector<int> local(G, -1);
    for (int i = 0; i < n; ++i) local[M[i]] = i;
    const int W = (n + 63) / 64;
    // dependencies inside the sub-graph
    std::vector<Mask> need(n, Mask(W, 0));
    bool free_choice = false;
    for (int i = 0; i < n; ++i)
      for (int d : deps[M[i]]) if (local[d] >= 0) mset(need[i], local[d]);
    // a chain has exactly one order: nothing to search
    for (int i = 1; i < n && !free_choice; ++i) if (!mtest(need[i], i - 1)) free_choice = true;
    if (!free_choice) { keep_default(); continue; }
    // roots seen from this sub-graph
    struct LRoot { Mask in; bool before, after; int64_t bytes[2]; };
    std::vector<LRoot> lr;
    std::vector<std::vector<int>> roots_of_group(n);
    for (const Root& R : roots) {
      LRoot L{Mask(W, 0), false, false, {R.bytes[0], R.bytes[1]}};
      bool here = false;
      for (int t : R.touch) {
        const int s = c->groups[t].subgraph;
        if (s < sg) L.before = true;
        else if (s > sg) L.after = true;
        else { mset(L.in, local[t]); here = true; }
      }
      if (!here) continue;
      for (int t : R.touch) if (local[t] >= 0) roots_of_group[local[t]].push_back(static_cast<int>(lr.size()));
      lr.push_back(std::move(L));
    }
    // level-by-level search over the down-closed sets
    std::vector<std::vector<Entry>> levels(n + 1);
    levels[0].push_back(Entry{Mask(W, 0), {INT64_MIN, INT64_MIN}, {0, 0}, -1, -1});
    size_t states = 1;
    bool abandoned = false;
    for (int lv = 0; lv < n && !abandoned; ++lv) {
      std::unordered_map<std::string, int> index;
      std::vector<Entry>& next = levels[lv + 1];
      for (int ei = 0; ei < static_cast<int>(levels[lv].size()) && !abandoned; ++ei) {
        for (int cand = 0; cand < n; ++cand) {
          const Entry& E = levels[lv][ei];
          if (mtest(E.mask, cand)) continue;
          bool ready = true;
          for (int w = 0; w < W; ++w) if (need[cand][w] & ~E.mask[w]) { ready = false; break; }
          if (!ready) continue;
          Mask nm = E.mask;
          mset(nm, cand);
          int64_t during[2] = {E.live[0], E.live[1]}, freed[2] = {0, 0};
          for (int ri : roots_of_group[cand]) {
            const LRoot& L = lr[ri];
            bool touched = L.before, remaining = L.after;
            for (int w = 0; w < W; ++w) {
              if (L.in[w] & E.mask[w]) touched = true;
              if (L.in[w] & ~nm[w]) remaining = true;
            }
            if (!touched) { during[0] += L.bytes[0]; during[1] += L.bytes[1]; }
            if (!remaining) { freed[0] += L.bytes[0]; freed[1] += L.bytes[1]; }
          }
          Entry N;
          for (int k = 0; k < 2; ++k) { N.peak[k] = std::max(E.peak[k], during[k]); N.live[k] = during[k] - freed[k]; }
          N.parent = ei;
          N.last = cand;
          const std::string key = mkey(nm);
          auto it = index.find(key);
          if (it == index.end()) {
            if (++states > STATE_BUDGET) { abandoned = true; break; }
            N.mask = std::move(nm);
            index.emplace(key, static_cast<int>(next.size()));
            next.push_back(std::move(N));
          } else if (better(N.peak, next[it->second].peak)) {
            Entry& X = next[it->second];
            X.peak[0] = N.peak[0]; X.peak[1] = N.peak[1];
            X.parent = N.parent; X.last = N.last;
          }
        }
      }
    }
    st.states += static_cast<int64_t>(states);
    if (abandoned || levels[n].empty()) { ++st.abandoned_subgraphs; keep_default(); continue; }
    ++st.searched_subgraphs;
    // the default order's peak inside this sub-graph, by the same accounting
    int64_t dpeak[2] = {INT64_MIN, INT64_MIN};
    {
      Mask m(W, 0);
      int64_t live[2] = {0, 0};
      for (int i = 0; i < n; ++i) {
        Mask nm = m;
        mset(nm, i);
        int64_t during[2] = {live[0], live[1]}, freed[2] = {0, 0};
        for (int ri : roots_of_group[i]) {
          const LRoot& L = lr[ri];
          bool touched = L.before, remaining = L.after;
          for (int w = 0; w < W; ++w) {
            if (L.in[w] & m[w]) touched = true;
            if (L.in[w] & ~nm[w]) remaining = true;
          }
          if (!touched) { during[0] += L.bytes[0]; during[1] += L.bytes[1]; }
          if (!remaining) { freed[0] += L.bytes[0]; freed[1] += L.bytes[1]; }
        }
        for (int k = 0; k < 2; ++k) { dpeak[k] = std::max(dpeak[k], during[k]); live[k] = during[k] - freed[k]; }
        m = nm;
      }
    }
    const Entry& F = levels[n][0];
    if (!better(F.peak, dpeak)) { keep_default(); continue; }
    std::vector<int> rev;
    int ei = 0;
    for (int lv = n; lv > 0; --lv) {
      const Entry& E = levels[lv][ei];
      rev.push_back(M[E.last]);
      ei = E.parent;
    }
    planned.insert(planned.end(), rev.rbegin(), rev.rend());
    ++st.reordered_subgraphs;
    any_change = true;
  }
  if (!any_change) return;
  int64_t ppeak[2];
  simulate(roots, planned, ppeak);
  // an improvement inside one sub-graph cannot raise the whole-graph peak; checked all the same
  if (better(st.default_peak, ppeak)) { st.reordered_subgraphs = 0; return; }
  st.planned_peak[0] = ppeak[0];
  st.planned_peak[1] = ppeak[1];
  *order = planned;
}

}  // namespace sod2
