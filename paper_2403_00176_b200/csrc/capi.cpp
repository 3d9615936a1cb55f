// C ABI (include/sod2.h) over the host core and the executor.
#include <cuda_runtime.h>

#include <cstring>
#include <list>
#include <new>
#include <unordered_map>

#include "../../include/sod2.h"
#include "engine.h"

using namespace sod2;

struct HandleBase {
  uint32_t magic;
  std::string err;
};
struct sod2_binding { HandleBase h{0x53443242u, ""}; Binding b; sod2_graph* g = nullptr; bool cached = false; };
struct sod2_plan_s { HandleBase h{0x53443250u, ""}; Plan p; sod2_graph* g = nullptr; bool cached = false; };
// Plan cache: binding + plan per bound symbol tuple, least recently used first out.  The entries belong
// to the graph; handles given out by sod2_plan_cached are borrowed.
struct PlanCacheEntry { std::string key; sod2_binding* b; sod2_plan_s* p; };
struct sod2_graph {
  HandleBase h{0x53443247u, ""};
  Compiled c;
  int cache_cap = 0;
  std::list<PlanCacheEntry> lru;                                             // front = most recently used
  std::unordered_map<std::string, std::list<PlanCacheEntry>::iterator> cache;
  void clear_cache() {
    for (auto& e : lru) { delete e.p; delete e.b; }
    lru.clear();
    cache.clear();
  }
  ~sod2_graph() { clear_cache(); }
};

static thread_local std::string g_create_err;

namespace sod2 {
void set_thread_error(const std::string& msg) { g_create_err = msg; }
}  // namespace sod2

static sod2_status st(Status s) { return static_cast<sod2_status>(s); }

static void copy_str(const std::string& s, char* buf, size_t len) {
  if (!buf || !len) return;
  size_t n = std::min(len - 1, s.size());
  std::memcpy(buf, s.data(), n);
  buf[n] = 0;
}

extern "C" {

const char* sod2_last_error(const void* h) {
  if (!h) return g_create_err.c_str();
  return static_cast<const HandleBase*>(h)->err.c_str();
}

sod2_status sod2_classify(const char* op, int* cls) {
  if (!op || !cls) return SOD2_E_INVALID_ARG;
  DynClass c;
  if (!classify_op(op, &c)) return SOD2_E_UNSUPPORTED_OP;
  *cls = static_cast<int>(c);
  return SOD2_OK;
}

sod2_status sod2_graph_create(const char* text, size_t len, uint32_t flags, sod2_graph** out) {
  if (!text || !out) { g_create_err = "null argument"; return SOD2_E_INVALID_ARG; }
  sod2_graph* g = new (std::nothrow) sod2_graph();
  if (!g) return SOD2_E_INTERNAL;
  g->c.flags = flags;
  Status s = parse_ir(text, len, &g->c.g);
  if (s == OK) s = rdp_analysis(&g->c.g);
  if (s != OK) { g_create_err = g->c.g.err; delete g; return st(s); }
  s = form_groups(&g->c);
  if (s != OK) { g_create_err = g->c.err; delete g; return st(s); }
  *out = g;
  return SOD2_OK;
}
void sod2_graph_destroy(sod2_graph* g) { delete g; }

sod2_status sod2_graph_reanalyse(sod2_graph* g, const int* order, int n) {
  if (!g || !order) return SOD2_E_INVALID_ARG;
  Graph& G = g->c.g;
  if (n != static_cast<int>(G.nodes.size())) { g->h.err = "order must list every operator once"; return SOD2_E_INVALID_ARG; }
  std::vector<int> ord(order, order + n), seen(n, 0);
  for (int v : ord) { if (v < 0 || v >= n || seen[v]) { g->h.err = "order is not a permutation"; return SOD2_E_INVALID_ARG; } seen[v] = 1; }
  // reset every produced tensor to undef, then iterate in the given order
  for (auto& t : G.tensors)
    if (t.producer >= 0) { t.S = ShapeVal(); t.V = ValueVal(); }
  G.asserts.clear();
  Status s = rdp_analysis(&G, &ord);
  if (s != OK) { g->h.err = G.err; return st(s); }
  g->c.groups.clear();
  g->c.packed_consts.clear(); g->c.packed_off.clear(); g->c.packed_ln.clear(); g->c.packed_bytes = 0;
  for (auto& nd : G.nodes) nd.group = -1;
  s = form_groups(&g->c);
  if (s != OK) g->h.err = g->c.err;
  return st(s);
}

sod2_status sod2_graph_set_const(sod2_graph* g, const char* name, const void* dev, size_t bytes) {
  if (!g || !name || !dev) return SOD2_E_INVALID_ARG;
  int t = g->c.g.tensor(name);
  if (t < 0 || g->c.g.tensors[t].kind != TKind::CONST) { g->h.err = std::string("no constant named ") + name; return SOD2_E_INVALID_ARG; }
  Tensor& T = g->c.g.tensors[t];
  size_t need = dtype_size(T.dtype);
  for (auto& d : T.S.dims) need *= static_cast<size_t>(d.e.const_value());
  if (bytes != need) { g->h.err = std::string("constant ") + name + ": expected " + std::to_string(need) + " bytes"; return SOD2_E_INVALID_ARG; }
  if (reinterpret_cast<uintptr_t>(dev) & 15) { g->h.err = "constants must be 16-byte aligned"; return SOD2_E_MISALIGNED; }
  T.dev_ptr = dev;
  T.dev_bytes = bytes;
  return SOD2_OK;
}

sod2_status sod2_graph_prepack_bytes(const sod2_graph* g, size_t* bytes) {
  if (!g || !bytes) return SOD2_E_INVALID_ARG;
  *bytes = g->c.packed_bytes;
  return SOD2_OK;
}
sod2_status sod2_graph_prepack(sod2_graph* g, void* ws, size_t bytes, void* stream) {
  if (!g) return SOD2_E_INVALID_ARG;
  Status s = prepack_weights(&g->c, ws, bytes, stream);
  if (s != OK) g->h.err = g->c.err;
  return st(s);
}

sod2_status sod2_bind_dims(sod2_graph* g, int n_req, int n_syms, const char* const* names, const int64_t* values, sod2_binding** out) {
  if (!g || !out || (n_syms > 0 && (!names || !values))) return SOD2_E_INVALID_ARG;
  sod2_binding* b = new (std::nothrow) sod2_binding();
  if (!b) return SOD2_E_INTERNAL;
  b->g = g;
  Status s = bind_dims(&g->c, n_req, n_syms, names, values, &b->b);
  if (s != OK) { g->h.err = b->b.err; delete b; return st(s); }
  *out = b;
  return SOD2_OK;
}
void sod2_binding_destroy(sod2_binding* b) { if (b && !b->cached) delete b; }

sod2_status sod2_plan(sod2_graph* g, const sod2_binding* b, sod2_plan_t** out, size_t* arena_bytes) {
  if (!g || !b || !out || b->g != g) return SOD2_E_INVALID_ARG;
  sod2_plan_s* p = new (std::nothrow) sod2_plan_s();
  if (!p) return SOD2_E_INTERNAL;
  p->g = g;
  Status s = make_plan(&g->c, &b->b, &p->p);
  if (s != OK) { g->h.err = p->p.err; delete p; return st(s); }
  if (arena_bytes) *arena_bytes = p->p.arena_bytes;
  *out = p;
  return SOD2_OK;
}
void sod2_plan_destroy(sod2_plan_t* p) { if (p && !p->cached) delete p; }

sod2_status sod2_graph_set_plan_cache(sod2_graph* g, int capacity) {
  if (!g || capacity < 0) return SOD2_E_INVALID_ARG;
  g->cache_cap = capacity;
  while (static_cast<int>(g->lru.size()) > capacity) {
    PlanCacheEntry& e = g->lru.back();
    g->cache.erase(e.key);
    delete e.p;
    delete e.b;
    g->lru.pop_back();
  }
  return SOD2_OK;
}

sod2_status sod2_plan_cached(sod2_graph* g, int n_req, int n_syms, const char* const* names, const int64_t* values,
                             sod2_binding** binding_out, sod2_plan_t** plan_out, size_t* arena_bytes, int* hit) {
  if (!g || !plan_out || n_req < 0 || n_syms < 0 || (n_syms > 0 && (!names || !values))) return SOD2_E_INVALID_ARG;
  if (g->cache_cap <= 0) { g->h.err = "the plan cache is disabled: call sod2_graph_set_plan_cache first"; return SOD2_E_INVALID_ARG; }
  std::string key(reinterpret_cast<const char*>(&n_req), sizeof n_req);
  for (int i = 0; i < n_syms; ++i) { key += names[i]; key.push_back('\0'); }
  key.append(reinterpret_cast<const char*>(values), static_cast<size_t>(n_req) * n_syms * sizeof(int64_t));
  auto it = g->cache.find(key);
  if (it != g->cache.end()) {
    g->lru.splice(g->lru.begin(), g->lru, it->second);   // most recently used
    if (hit) *hit = 1;
  } else {
    sod2_binding* b = new (std::nothrow) sod2_binding();
    sod2_plan_s* p = new (std::nothrow) sod2_plan_s();
    if (!b || !p) { delete b; delete p; return SOD2_E_INTERNAL; }
    b->g = g; b->cached = true;
    p->g = g; p->cached = true;
    Status s = bind_dims(&g->c, n_req, n_syms, names, values, &b->b);
    if (s != OK) { g->h.err = b->b.err; delete b; delete p; return st(s); }
    s = make_plan(&g->c, &b->b, &p->p);
    if (s != OK) { g->h.err = p->p.err; delete p; delete b; return st(s); }
    if (static_cast<int>(g->lru.size()) >= g->cache_cap) {
      PlanCacheEntry& e = g->lru.back();
      g->cache.erase(e.key);
      delete e.p;
      delete e.b;
      g->lru.pop_back();
    }
    g->lru.push_front(PlanCacheEntry{key, b, p});
    g->cache[key] = g->lru.begin();
    if (hit) *hit = 0;
  }
  PlanCacheEntry& e = g->lru.front();
  if (binding_out) *binding_out = e.b;
  *plan_out = e.p;
  if (arena_bytes) *arena_bytes = e.p->p.arena_bytes;
  return SOD2_OK;
}

sod2_status sod2_run(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes,
                     void* stream, sod2_run_info* info) {
  if (!p || !inputs || !outputs) return SOD2_E_INVALID_ARG;
  const Graph& G = p->g->c.g;
  for (size_t i = 0; i < G.inputs.size(); ++i) if (!inputs[i]) { p->h.err = "null input"; return SOD2_E_INVALID_ARG; }
  for (size_t i = 0; i < G.outputs.size(); ++i) if (!outputs[i]) { p->h.err = "null output"; return SOD2_E_INVALID_ARG; }
  if (arena_bytes < p->p.arena_bytes) { p->h.err = "arena too small"; return SOD2_E_ARENA_TOO_SMALL; }
  if (reinterpret_cast<uintptr_t>(arena) & 255) { p->h.err = "arena must be 256-byte aligned"; return SOD2_E_MISALIGNED; }
  for (int c : G.consts) {
    bool used = false;
    for (auto& grp : p->g->c.groups) for (int t : grp.ext_in) if (t == c) used = true;
    if (used && !G.tensors[c].dev_ptr) { p->h.err = "constant " + G.tensors[c].name + " has no device data"; return SOD2_E_INVALID_ARG; }
  }
  int64_t inf[8] = {0};
  Status s = run_plan(&p->p, inputs, outputs, arena, arena_bytes, stream, inf);
  if (s != OK) p->h.err = p->p.err;
  if (info) { info->host_enqueue_ns = inf[0]; info->gpu_launches = inf[1]; }
  return st(s);
}

sod2_status sod2_run_graph(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes,
                           void* stream, sod2_run_info* info) {
  if (!p || !inputs || !outputs) return SOD2_E_INVALID_ARG;
  const Graph& G = p->g->c.g;
  for (size_t i = 0; i < G.inputs.size(); ++i) if (!inputs[i]) { p->h.err = "null input"; return SOD2_E_INVALID_ARG; }
  for (size_t i = 0; i < G.outputs.size(); ++i) if (!outputs[i]) { p->h.err = "null output"; return SOD2_E_INVALID_ARG; }
  for (int c : G.consts) {
    bool used = false;
    for (auto& grp : p->g->c.groups) for (int t : grp.ext_in) if (t == c) used = true;
    if (used && !G.tensors[c].dev_ptr) { p->h.err = "constant " + G.tensors[c].name + " has no device data"; return SOD2_E_INVALID_ARG; }
  }
  int64_t inf[8] = {0};
  Status s = run_plan_graph(&p->p, inputs, outputs, arena, arena_bytes, stream, inf);
  if (s != OK) p->h.err = p->p.err;
  if (info) { info->host_enqueue_ns = inf[0]; info->gpu_launches = inf[1]; info->reserved[1] = inf[3]; }
  return st(s);
}

sod2_status sod2_run_exact(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes,
                           void* stream, sod2_run_info* info) {
  if (!p || !inputs || !outputs || !arena) return SOD2_E_INVALID_ARG;
  if (arena_bytes < p->p.arena_bytes) { p->h.err = "arena too small"; return SOD2_E_ARENA_TOO_SMALL; }
  if (reinterpret_cast<uintptr_t>(arena) & 255) { p->h.err = "arena must be 256-byte aligned"; return SOD2_E_MISALIGNED; }
  if (p->g->c.packed_bytes && !p->g->c.packed_ws) { p->h.err = "weights are not prepacked"; return SOD2_E_INVALID_ARG; }
  if (!p->p.sm_count_known) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) p->p.sm_count = n;
    p->p.sm_count_known = true;
  }
  int64_t inf[8] = {0};
  std::string err;
  Status s = run_exact(&p->g->c, p->p.b, &p->p, inputs, outputs, arena, arena_bytes, stream, inf, &err);
  if (s != OK) p->h.err = err;
  if (info) {
    info->host_enqueue_ns = inf[0]; info->gpu_launches = inf[1];
    info->reserved[2] = inf[2]; info->reserved[3] = inf[3]; info->reserved[4] = inf[4];
  }
  return st(s);
}

sod2_status sod2_plan_poison_arena(sod2_plan_t* p, void* arena, size_t arena_bytes, void* stream) {
  if (!p || !arena) return SOD2_E_INVALID_ARG;
  Status s = poison_arena(&p->p, arena, arena_bytes, stream);
  if (s != OK) p->h.err = s == E_ARENA_TOO_SMALL ? "arena too small" : "cannot fill the arena";
  return st(s);
}

sod2_status sod2_plan_check_guards(sod2_plan_t* p, void* arena, void* stream, int* n_damaged, char* first_name, size_t first_name_len) {
  if (!p || !arena || !n_damaged) return SOD2_E_INVALID_ARG;
  if (!(p->g->c.flags & OPT_GUARD_BANDS)) { p->h.err = "the graph was not created with SOD2_OPT_GUARD_BANDS"; return SOD2_E_INVALID_ARG; }
  int bad = 0, first = -3;
  Status s = check_guards(&p->p, arena, stream, &bad, &first);
  if (s != OK) { p->h.err = "cannot check the guard bands"; return st(s); }
  *n_damaged = bad;
  copy_str(first >= 0 ? p->g->c.g.tensors[first].name : first == -1 ? "<group scratch>" : first == -2 ? "<index lists>" : "", first_name, first_name_len);
  return SOD2_OK;
}

sod2_status sod2_run_timed(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes,
                           void* stream, float* group_ms, int n_groups) {
  if (!p || !inputs || !outputs || !arena) return SOD2_E_INVALID_ARG;
  Status s = run_plan_timed(&p->p, inputs, outputs, arena, arena_bytes, stream, group_ms, n_groups);
  if (s != OK) p->h.err = p->p.err;
  return st(s);
}

sod2_status sod2_run_timed_repeat(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes,
                                  void* stream, int reps, float* group_ms, int n_groups) {
  if (!p || !inputs || !outputs || !arena) return SOD2_E_INVALID_ARG;
  Status s = run_plan_timed(&p->p, inputs, outputs, arena, arena_bytes, stream, group_ms, n_groups, reps);
  if (s != OK) p->h.err = p->p.err;
  return st(s);
}

sod2_status sod2_plan_device_status(sod2_plan_t* p, const void* arena, void* stream) {
  if (!p || !arena) return SOD2_E_INVALID_ARG;
  int word = 0;
  if (!p->p.uses_header) {   // no kernel of this plan has a bounded wait: the word is never written (nor cleared)
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { p->h.err = "cannot synchronise the stream"; return SOD2_E_CUDA; }
    return SOD2_OK;
  }
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess ||
      cudaMemcpy(&word, arena, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    p->h.err = "cannot read the device status word";
    return SOD2_E_CUDA;
  }
  if (word) { p->h.err = "a kernel gave up on a bounded wait"; return SOD2_E_TIMEOUT; }
  return SOD2_OK;
}

// ---------------------------------------------------------------- introspection
sod2_status sod2_graph_tensor_info(const sod2_graph* g, const char* name, int* rank, int* dim_kind, char* buf, size_t len) {
  if (!g || !name) return SOD2_E_INVALID_ARG;
  int t = g->c.g.tensor(name);
  if (t < 0) return SOD2_E_INVALID_ARG;
  const Graph& G = g->c.g;
  const ShapeVal& s = G.tensors[t].S;
  if (rank) *rank = s.rank;
  if (dim_kind)
    for (int i = 0; i < s.rank; ++i) {
      const Dim& d = s.dims[i];
      int k = 0;
      if (d.kind == Dim::NAC) k = 4;
      else if (d.kind == Dim::VAL) k = e_has_runtime(G.cx, d.e) ? 4 : d.e.is_const() ? 1 : d.e.is_symbol() ? 2 : 3;
      dim_kind[i] = k;
    }
  copy_str(shape_str(G, s), buf, len);
  return SOD2_OK;
}

sod2_status sod2_graph_tensor_dtype(const sod2_graph* g, const char* name, int* dtype) {
  if (!g || !name || !dtype) return SOD2_E_INVALID_ARG;
  int t = g->c.g.tensor(name);
  if (t < 0) return SOD2_E_INVALID_ARG;
  *dtype = static_cast<int>(g->c.g.tensors[t].dtype);
  return SOD2_OK;
}

sod2_status sod2_graph_tensor_value(const sod2_graph* g, const char* name, char* buf, size_t len) {
  if (!g || !name) return SOD2_E_INVALID_ARG;
  int t = g->c.g.tensor(name);
  if (t < 0) return SOD2_E_INVALID_ARG;
  const ValueVal& v = g->c.g.tensors[t].V;
  if (v.kind == ValueVal::UNDEF) copy_str("undef", buf, len);
  else if (v.kind == ValueVal::NAC) copy_str("nac", buf, len);
  else { ShapeVal s; s.rank = static_cast<int>(v.elems.size()); s.dims = v.elems; copy_str(shape_str(g->c.g, s), buf, len); }
  return SOD2_OK;
}

int sod2_graph_num_ops(const sod2_graph* g) { return g ? static_cast<int>(g->c.g.nodes.size()) : -1; }
int sod2_graph_num_groups(const sod2_graph* g) { return g ? static_cast<int>(g->c.groups.size()) : -1; }
int sod2_graph_num_subgraphs(const sod2_graph* g) { return g ? g->c.n_subgraphs : -1; }
int sod2_graph_rdp_sweeps(const sod2_graph* g) { return g ? g->c.g.rdp_sweeps : -1; }

sod2_status sod2_graph_order_info(const sod2_graph* g, int64_t* out) {
  if (!g || !out) return SOD2_E_INVALID_ARG;
  const OrderStats& s = g->c.order_stats;
  out[0] = s.default_peak[0]; out[1] = s.default_peak[1];
  out[2] = s.planned_peak[0]; out[3] = s.planned_peak[1];
  out[4] = s.states;
  out[5] = s.searched_subgraphs; out[6] = s.reordered_subgraphs; out[7] = s.abandoned_subgraphs;
  out[8] = s.unbounded;
  return SOD2_OK;
}

sod2_status sod2_graph_op_info(const sod2_graph* g, int op, char* type, size_t type_len, int* cls, int* eff, int* group, int* sub) {
  if (!g || op < 0 || op >= static_cast<int>(g->c.g.nodes.size())) return SOD2_E_INVALID_ARG;
  const Node& n = g->c.g.nodes[op];
  copy_str(n.op, type, type_len);
  if (cls) *cls = static_cast<int>(n.cls);
  if (eff) *eff = static_cast<int>(n.eff_cls);
  if (group) *group = n.group;
  if (sub) *sub = n.subgraph;
  return SOD2_OK;
}

sod2_status sod2_graph_group_info(const sod2_graph* g, int gi, char* kind, size_t kind_len, int* n_ops, int* versions, int* sub) {
  if (!g || gi < 0 || gi >= static_cast<int>(g->c.groups.size())) return SOD2_E_INVALID_ARG;
  const Group& G = g->c.groups[gi];
  copy_str(gkind_name(G.kind), kind, kind_len);
  if (n_ops) *n_ops = static_cast<int>(G.nodes.size());
  if (versions) *versions = G.versions;
  if (sub) *sub = G.subgraph;
  return SOD2_OK;
}

sod2_status sod2_binding_shape(const sod2_binding* b, int r, const char* name, int64_t* dims, int* rank) {
  if (!b || !name || r < 0 || r >= b->b.n_req) return SOD2_E_INVALID_ARG;
  int t = b->g->c.g.tensor(name);
  if (t < 0) return SOD2_E_INVALID_ARG;
  if (b->b.dims[t].empty()) return SOD2_E_UNBOUND_SYMBOL;
  const auto& d = b->b.dims[t][r];
  if (rank) *rank = static_cast<int>(d.size());
  if (dims) for (size_t i = 0; i < d.size(); ++i) dims[i] = d[i];
  return SOD2_OK;
}

sod2_status sod2_plan_slot(const sod2_plan_t* p, const char* name, size_t* off, size_t* bytes, int* def, int* last) {
  if (!p || !name) return SOD2_E_INVALID_ARG;
  int t = p->g->c.g.tensor(name);
  if (t < 0 || p->p.views[t].empty() || p->p.root_of[t] < 0) return SOD2_E_INVALID_ARG;
  if (p->p.root_of[t] != t) return SOD2_E_INVALID_ARG;  // a view: it owns no slot
  const RootBuf& R = p->p.roots[t];
  if (R.where != RootBuf::ARENA) return SOD2_E_INVALID_ARG;
  if (off) *off = R.arena_off;
  if (bytes) *bytes = static_cast<size_t>(R.bytes);
  if (def) *def = R.def_step;
  if (last) *last = R.last_step;
  return SOD2_OK;
}

sod2_status sod2_plan_instance_offset(const sod2_plan_t* p, const char* name, int r, size_t* off) {
  if (!p || !name || !off || r < 0 || r >= p->p.n_req) return SOD2_E_INVALID_ARG;
  int t = p->g->c.g.tensor(name);
  if (t < 0 || p->p.views[t].empty() || p->p.root_of[t] < 0) return SOD2_E_INVALID_ARG;
  const View& v = p->p.views[t][r];
  *off = static_cast<size_t>(p->p.inst_off[p->p.root_of[t]][r] + v.offset * dtype_size(p->g->c.g.tensors[t].dtype));
  return SOD2_OK;
}

sod2_status sod2_plan_tensor_strides(const sod2_plan_t* p, const char* name, int r, int64_t* strides, int* rank) {
  if (!p || !name || r < 0 || r >= p->p.n_req) return SOD2_E_INVALID_ARG;
  int t = p->g->c.g.tensor(name);
  if (t < 0 || p->p.views[t].empty() || p->p.root_of[t] < 0) return SOD2_E_INVALID_ARG;
  const View& v = p->p.views[t][r];
  if (rank) *rank = static_cast<int>(v.strides.size());
  if (strides) for (size_t i = 0; i < v.strides.size(); ++i) strides[i] = v.strides[i];
  return SOD2_OK;
}

sod2_status sod2_plan_group_cost(const sod2_plan_t* p, int group, double* flops, double* bytes) {
  if (!p || group < 0 || group >= static_cast<int>(p->p.group_flops.size())) return SOD2_E_INVALID_ARG;
  if (flops) *flops = p->p.group_flops[group];
  if (bytes) *bytes = p->p.group_bytes[group];
  return SOD2_OK;
}

sod2_status sod2_plan_group_on_side_stream(const sod2_plan_t* p, int group, int* on_side) {
  if (!p || !on_side || group < 0 || group >= static_cast<int>(p->p.side_group.size())) return SOD2_E_INVALID_ARG;
  *on_side = p->p.side_group[group] ? 1 : 0;
  return SOD2_OK;
}

sod2_status sod2_plan_memory(const sod2_plan_t* p, size_t* arena, size_t* peak, size_t* sum) {
  if (!p) return SOD2_E_INVALID_ARG;
  if (arena) *arena = p->p.arena_bytes;
  if (peak) *peak = p->p.peak_live_bytes;
  if (sum) *sum = p->p.sum_bytes;
  return SOD2_OK;
}

sod2_status sod2_run_output_shape(sod2_plan_t* p, const void* arena, void* stream, int r, int output, int64_t* dims, int* rank) {
  if (!p || r < 0 || r >= p->p.n_req) return SOD2_E_INVALID_ARG;
  const Graph& G = p->g->c.g;
  if (output < 0 || output >= static_cast<int>(G.outputs.size())) return SOD2_E_INVALID_ARG;
  const Tensor& T = G.tensors[G.outputs[output]];
  if (T.S.rank < 0) return SOD2_E_INTERNAL;
  std::vector<int64_t> vals = p->p.b->vals[r];
  bool need = false;
  for (auto& d : T.S.dims) if (d.known() && e_has_runtime(G.cx, d.e)) need = true;
  if (need) {
    if (!arena) return SOD2_E_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SOD2_E_CUDA;
    for (size_t a = 0; a < G.cx.atoms.size(); ++a) {
      if (G.cx.atoms[a].kind != AtomKind::SYM || !G.cx.atoms[a].runtime) continue;
      long long v = 0;
      const char* src = static_cast<const char*>(arena) + 256 + (a * p->p.n_req + r) * 8;
      if (cudaMemcpy(&v, src, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return SOD2_E_CUDA;
      vals[a] = v;
    }
  }
  if (rank) *rank = T.S.rank;
  for (int i = 0; i < T.S.rank; ++i) {
    bool ok;
    int64_t v = e_eval(G.cx, T.S.dims[i].e, vals, &ok);
    if (!ok) return SOD2_E_UNBOUND_SYMBOL;
    if (dims) dims[i] = v;
  }
  return SOD2_OK;
}

}  // extern "C"
