// Fused groups, per-request binding, arena memory plan and launch plan.
#pragma once
#include <initializer_list>
#include <memory>
#include <new>
#include <string>
#include <type_traits>
#include <vector>

#include "graph.h"

namespace sod2 {

enum OptFlags : uint32_t {
  OPT_NO_FUSION = 1u,   // every operator is its own group (fused-vs-unfused comparison)
  OPT_NO_REUSE = 2u,    // every arena tensor gets its own slot (keeps all intermediates readable after a run)
  OPT_COPY_REGROUP = 16u,     // Switch / Combine always move whole samples (no index-indirect convolutions)
  OPT_LEGACY_ATTENTION = 8u,  // attention groups on the mma.sync kernel even where the tcgen05 kernel applies
  OPT_MULTI_VERSION = 64u,    // fuse elementwise chains across unresolved broadcasts: 2^d versions, chosen at bind time
  OPT_NO_SEP = 32u,     // groups run in their default topological order (no static execution planning)
  OPT_SPLITK_LN = 4u,   // a bf16 GEMM (+bias, +residual) followed by LayerNorm becomes one group: split-K GEMM + finishing kernel
  OPT_LN_FOLD = 128u,     // a LayerNorm between bf16 GEMMs is folded into their epilogues (the normalised tensor is never stored)
  OPT_GUARD_BANDS = 512u, // 256 poison bytes behind every arena tensor and scratch region, checked after a run (sod2_plan_check_guards)
  OPT_GEMM_PAIR = 1024u,  // bf16 GEMMs on CTA pairs (tcgen05.mma.cta_group::2) where the makespan estimate favours them
  OPT_GEMM_CHAIN = 256u,  // consecutive dependent GEMM groups run as one persistent kernel with row-block dependency counters
};

enum class GKind {
  GEMM,        // MatMul(x, const W) [+bias] [act] [+residual]          (tcgen05, bf16) or the fp32 SIMT kernel [+LayerNorm]
  ATTENTION,   // MatMul(q,k^T) [*scale] Softmax MatMul(p,v)
  LAYERNORM,   // LayerNormalization alone on packed rows
  CHAIN,       // broadcast-elementwise chain [+ trailing Softmax / LayerNormalization]
  TOPK_KEEP,   // ReduceSumSquare -> TopK(order=index) -> Gather rows
  NONZERO,
  CONV,        // Conv [+bias] [act] [+residual] [act]
  GAP,         // GlobalAveragePool
  GATE,        // GlobalAveragePool -> Reshape -> MatMul(C x 1) -> Add -> Greater
  SWITCH,
  COMBINE,
  LAYOUT,      // NCHW <-> channels-last storage change at the ABI boundary of convolution graphs (act: 0 to, 1 from)
  // stand-alone forms of operators that otherwise run inside fused groups (unfused mode, or outside their pattern)
  BMM,         // MatMul of two activations (batched, strided operands)
  SUMSQ,       // ReduceSumSquare over the last axis
  TOPK,        // TopK over the last axis: values + int64 indices
  GATHER,      // Gather along one axis by an int64 index tensor computed on the device
  FILL,        // Range / ConstantOfShape whose extent is only known at bind time: out[i] = start + i * step
  RESIZE,      // Resize / Upsample, nearest neighbour: out[.., o, ..] = x[.., floor(o * in / out), ..]
  UNSUPPORTED
};
const char* gkind_name(GKind k);

struct Group {
  GKind kind = GKind::UNSUPPORTED;
  std::vector<int> nodes;
  std::vector<int> ext_in, ext_out;   // tensors crossing the group boundary
  int versions = 1;                   // fused code versions needed (2^unresolved broadcast dims, Section 4.2)
  int subgraph = 0;
  // roles (tensor ids, -1 = absent)
  int a = -1, w = -1, bias = -1, res = -1, out = -1, gamma = -1, beta = -1;
  int q = -1, k = -1, v = -1, out2 = -1, gate = -1;
  int act = 0;                        // 0 none, 1 gelu, 2 relu
  int act2 = 0;                       // activation after the residual add
  int has_ln = 0;
  int red = 0;                        // chain: 0 none, 1 softmax, 2 layernorm
  float eps = 1e-5f, scale = 1.0f;
  int stride = 1, pad = 0, ksize = 1;
  // LayerNorm folded into the neighbouring GEMMs (fuse.cpp, step 3c): the normalised tensor is never stored.
  //   ln_a >= 0:   the A operand is LayerNorm(ln_a): the kernel multiplies the raw rows by gamma-scaled weights and
  //                its epilogue applies the rows' mean / rstd and two precomputed vectors
  //   ln_res >= 0: the residual operand is LayerNorm(ln_res): the epilogue normalises the staged raw tile
  //   emit_stats:  the epilogue also writes per-row partial statistics of the output (beside the output's storage)
  int ln_a = -1, ln_res = -1, ln_gamma = -1, ln_beta = -1, emit_stats = 0;
  float ln_eps = 1e-5f;
  std::vector<int> chain_ops;         // ChainOp codes
  std::vector<int> chain_operands;    // tensor id or -1 per op
  std::string why;                    // for UNSUPPORTED
};

// How a tensor's storage relates to others (decided once, at graph creation).
struct Storage {
  // INDIRECT_IN: an output of a Switch that is never copied: the samples of the Switch input selected
  // by the executed / skipped id list.  INDIRECT_OUT: the executed operand of a Combine, written by its
  // producer straight into the Combine output at the executed ids.
  // ALIAS: the tensor lives in the storage of `other` (same extents): the output of a Combine whose
  // skipped samples are already where they belong, because the executed ones are written in place.
  enum Kind { ROOT, VIEW_OF_INPUT, VIEW_OF_OUTPUT, FOLDED, INDIRECT_IN, INDIRECT_OUT, ALIAS } kind = ROOT;
  int node = -1;    // the view operator (Switch / Combine for the indirect kinds)
  int other = -1;   // VIEW_OF_INPUT / INDIRECT_IN: the operator's input; VIEW_OF_OUTPUT / INDIRECT_OUT: the operator's output
  int gate = -1;    // indirect kinds: the gate tensor whose partition gives the id lists
  int list = 0;     // indirect kinds: 0 = executed ids, 1 = skipped ids
};

// Outcome of static execution planning (Section 4.3): peak of live arena bytes of the default and of
// the planned group order, at the upper [0] and lower [1] corner of the declared symbol ranges.
struct OrderStats {
  int64_t default_peak[2] = {0, 0}, planned_peak[2] = {0, 0};
  int64_t states = 0;                 // sets of finished groups visited by the search
  int searched_subgraphs = 0, reordered_subgraphs = 0, abandoned_subgraphs = 0;
  int unbounded = 0;                  // 1: some tensor size has no static bound, nothing was searched
};

struct Compiled {
  Graph g;
  OrderStats order_stats;
  uint32_t flags = 0;
  std::vector<Group> groups;          // in execution order
  std::vector<Storage> storage;       // per tensor
  std::vector<int> node_folded;       // per node: 1 = evaluated by RDP (shape arithmetic) or a pure view
  int n_subgraphs = 1;
  // prepacked (transposed, K-major) copies of GEMM weights
  // every distinct extent expression once: binding evaluates each per request, tensors index the table
  std::vector<Expr> dim_exprs;
  std::vector<std::vector<int>> dim_expr_id;   // [tensor][axis] -> dim_exprs index, -1 if the extent is unknown
  // Shape classes: tensors of one dim_class have the same extent expressions axis by axis; tensors of one view_class
  // resolve to the same offsets, extents and strides for every binding (same storage kind, same class of the tensor
  // they are derived from, same view parameters, same element size and layout rule).  Binding and planning fill
  // one table row per class and let the other members read it.
  std::vector<int> dim_class, view_class;
  int n_dim_classes = 0, n_view_classes = 0;
  // per tensor stored as a view: the operator's parameters read out of its attributes once (Transpose:
  // a = perm; Slice: a = start, b = step per axis of the input), so that planning touches no strings
  struct ViewParam { int op = -1; std::vector<int64_t> a, b; };   // op: 0 Transpose, 1 Reshape, 2 Slice
  std::vector<ViewParam> view_param;
  std::vector<int> packed_consts;     // tensor ids
  std::vector<size_t> packed_off;     // byte offsets in the prepack workspace
  // entry i with packed_ln[i].gamma >= 0 is the weight of a GEMM whose A operand is a folded LayerNorm:
  // [N,K] bf16 copy of gamma[k] * W[k,n], then fp32 c1[N] = column sums of that copy, then fp32
  // c2[N] = sum_k beta[k] * W[k,n] + bias[n]
  struct PackedLn { int gamma = -1, beta = -1, bias = -1; };
  std::vector<PackedLn> packed_ln;
  // per tensor: > 0 = row width of a tensor whose producer writes LayerNorm row statistics beside it
  std::vector<int> stats_width;
  size_t packed_bytes = 0;
  void* packed_ws = nullptr;
  std::string err;
};

// Message returned by sod2_last_error(NULL) on the calling thread (errors of calls without a handle).
void set_thread_error(const std::string& msg);

Status form_groups(Compiled* c);
// Static execution planning: `order` (default topological order on entry) becomes the order of least
// peak live bytes found per sub-graph; deps[g] lists the groups that must precede g.
void plan_execution_order(Compiled* c, const std::vector<std::vector<int>>& deps, std::vector<int>* order);
// Transposed (K-major) copies of the GEMM weights into caller-owned workspace; enqueued on `stream`.
Status prepack_weights(Compiled* c, void* workspace, size_t bytes, void* stream);

// ---- per-request binding (H0: substitute symbol values into every expression)
// Extents or strides of one tensor instance, stored inline: binding and planning create one per
// (tensor, request) and a heap vector for each was most of their cost.
constexpr int MAX_RANK = 8;
struct DimVec {
  int64_t v[MAX_RANK];
  int n = 0;
  DimVec() {}
  DimVec(std::initializer_list<int64_t> l) { for (auto x : l) v[n++] = x; }
  DimVec(size_t count, int64_t val) : n(static_cast<int>(count)) { for (int i = 0; i < n; ++i) v[i] = val; }
  size_t size() const { return static_cast<size_t>(n); }
  bool empty() const { return n == 0; }
  int64_t& operator[](size_t i) { return v[i]; }
  const int64_t& operator[](size_t i) const { return v[i]; }
  int64_t* begin() { return v; }
  int64_t* end() { return v + n; }
  const int64_t* begin() const { return v; }
  const int64_t* end() const { return v + n; }
  int64_t back() const { return v[n - 1]; }
  void resize(size_t k, int64_t val = 0) { for (int i = n; i < static_cast<int>(k); ++i) v[i] = val; n = static_cast<int>(k); }
  void assign(size_t k, int64_t val) { n = static_cast<int>(k); for (int i = 0; i < n; ++i) v[i] = val; }
  void push_back(int64_t x) { v[n++] = x; }
  bool operator==(const DimVec& o) const { if (n != o.n) return false; for (int i = 0; i < n; ++i) if (v[i] != o.v[i]) return false; return true; }
  bool operator!=(const DimVec& o) const { return !(*this == o); }
};

// Blocks of host memory for the per-batch tables, recycled between plans: a table of a batch is one to two
// megabytes, and a fresh allocation of that size is mapped page by page on first touch, which cost more than filling
// it.  block_acquire returns at least `need` bytes (the capacity in *cap); block_release hands the block back.
unsigned char* block_acquire(size_t need, size_t* cap);
void block_release(unsigned char* p, size_t cap);

// [tensor][request] table in one block of memory: binding and planning fill a few thousand small entries per
// batch, and one vector per tensor made the allocator the largest cost of both.  A row exists once make(t) was
// called; the others read as empty.  A row made with make_shared holds ONE entry that every request index reads
// (constants, and anything whose extents are equal for all requests of the batch); alias(t, rep) makes a tensor read
// another tensor's row (tensors of one shape class: most of a model's tensors repeat a handful of shapes).  T must
// be trivially destructible (nothing is destroyed).
template <class T>
class ReqTable {
 public:
  template <class U>
  class RowT {
   public:
    RowT(U* p, int n, int stride) : p_(p), n_(n), stride_(stride) {}
    bool empty() const { return n_ == 0; }
    size_t size() const { return static_cast<size_t>(n_); }
    U& operator[](size_t r) const { return p_[r * stride_]; }
    bool shared() const { return stride_ == 0; }
   private:
    U* p_;
    int n_;
    int stride_;   // 0: one entry stands for every request
  };
  using Row = RowT<T>;
  using ConstRow = RowT<const T>;
  void reset(size_t n_tensors, int n_req) {
    static_assert(std::is_trivially_destructible<T>::value, "rows are never destroyed");
    n_req_ = n_req;
    has_.assign(n_tensors, 0);
    at_.resize(n_tensors);
    const size_t need = n_tensors * static_cast<size_t>(n_req) * sizeof(T);
    if (need > cap_) { release(); raw_ = block_acquire(need, &cap_); }
  }
  ReqTable() {}
  ReqTable(const ReqTable&) = delete;
  ReqTable& operator=(const ReqTable&) = delete;
  ~ReqTable() { release(); }
  // a row with one entry per request
  Row make(size_t t) {
    if (!has_[t]) { at_[t] = static_cast<int>(t); T* p = slot(t); for (int r = 0; r < n_req_; ++r) new (p + r) T(); has_[t] = 1; }
    return (*this)[t];
  }
  // a row whose single entry is what every request reads (the value does not depend on the request in this batch)
  Row make_shared(size_t t) {
    if (!has_[t]) { at_[t] = static_cast<int>(t); new (slot(t)) T(); has_[t] = 2; }
    return (*this)[t];
  }
  // tensor t reads the row of tensor `rep` (same content by construction): nothing is copied
  void alias(size_t t, size_t rep) { at_[t] = at_[rep]; has_[t] = has_[rep]; }
  bool shared(size_t t) const { return has_[t] == 2; }
  Row operator[](size_t t) { return has_[t] ? Row(slot(t), n_req_, has_[t] == 2 ? 0 : 1) : Row(nullptr, 0, 1); }
  ConstRow operator[](size_t t) const { return has_[t] ? ConstRow(slot(t), n_req_, has_[t] == 2 ? 0 : 1) : ConstRow(nullptr, 0, 1); }
  size_t size() const { return has_.size(); }
 private:
  T* slot(size_t t) const { return reinterpret_cast<T*>(raw_) + static_cast<size_t>(at_[t]) * n_req_; }
  void release() { if (raw_) block_release(raw_, cap_); raw_ = nullptr; cap_ = 0; }
  unsigned char* raw_ = nullptr;
  size_t cap_ = 0;
  std::vector<char> has_;
  std::vector<int> at_;     // which tensor's slot holds the row (its own unless aliased)
  int n_req_ = 0;
};

struct Binding {
  const Compiled* c = nullptr;
  int n_req = 0;
  std::vector<std::vector<int64_t>> vals;   // [req][atom]
  ReqTable<DimVec> dims;                    // [tensor][req]; empty if not evaluable yet
  std::string err;
};
Status bind_dims(const Compiled* c, int n_req, int n_syms, const char* const* names, const int64_t* values, Binding* out);
Status evaluate_dims(Binding* out);
Status rebind_runtime(const Binding& base, const std::vector<std::vector<std::pair<int, int64_t>>>& rt_vals, Binding* out);

// ---- plan
struct View {                 // one tensor of one request, resolved to storage (which tensor owns the bytes: Plan::root_of)
  int64_t offset = 0;         // elements from the start of the root's instance for this request
  DimVec dims, strides;       // elements
  int ind_gate = -1;          // >= 0: sample n of this tensor is sample ids[n] of the root (ids = list `ind_list` of that gate's partition)
  int ind_list = 0;
  bool contiguous() const {
    int64_t s = 1;
    for (int i = static_cast<int>(dims.size()) - 1; i >= 0; --i) { if (dims[i] != 1 && strides[i] != s) return false; s *= dims[i]; }
    return true;
  }
};

struct RootBuf {              // packed storage of a root tensor: the requests' instances back to back
  enum Where { NONE, INPUT, OUTPUT, CONST, ARENA } where = NONE;
  int io_index = -1;
  int64_t bytes = 0;
  size_t arena_off = 0;
  int def_step = -1, last_step = -1;
  // LayerNorm row statistics written by the producing GEMM (folded LayerNorm): `stats_slots` planes of
  // `stats_rows` (mean, M2) float pairs at byte `stats_off` of this root's storage, one pair per packed row
  int64_t stats_off = -1, stats_rows = 0;
  int stats_slots = 0;
};

struct Ptr {                  // address resolved at run time
  int where = 0;              // RootBuf::Where, or 5 = prepack workspace, 6 = scratch in arena
  int index = -1;
  int64_t off = 0;
};

struct Launch;                // defined in exec.cu

struct Plan {
  const Compiled* c = nullptr;
  const Binding* b = nullptr;
  int n_req = 0;
  ReqTable<View> views;                   // [tensor][req]
  std::vector<int> root_of;               // [tensor] id of the tensor that owns the bytes (-1: not resolved)
  ReqTable<int64_t> inst_off;             // [root tensor][req] byte offset of the request's instance in the root's packed storage
  std::vector<RootBuf> roots;             // [tensor]
  size_t arena_bytes = 0, peak_live_bytes = 0, sum_bytes = 0;
  int peak_step = 0;
  std::vector<std::shared_ptr<Launch>> launches;
  std::vector<size_t> scratch_off;        // per group scratch offsets in the arena
  int gpu_launches = 0;
  int sm_count = 148;                     // persistent kernels launch one CTA per SM
  bool sm_count_known = false;
  bool uses_header = true;                // false: no kernel of the plan writes the status word, a ticket or a count: nothing to clear or read
  std::vector<double> group_flops, group_bytes;   // algorithmic cost per group for the bound shapes
  // per tensor with row statistics: slots the producer's tile version really writes and columns per slot
  struct StatsLayout { int slots = 0, cols = 0; };
  std::vector<StatsLayout> stats_layout;
  // Runs of consecutive GEMM groups that execute as one persistent kernel (gemm_chain_tcgen05.cuh): decided after
  // view resolution and before liveness, because the members run concurrently: everything a member reads stays
  // live, and everything a member writes is live, over the whole run.
  struct Chain { std::vector<int> groups; int rows = 0; size_t counter_word = 0; };
  std::vector<Chain> chains;
  std::vector<int> chain_of;              // [group] index into chains, -1 = a launch of its own
  size_t chain_counter_off = 0;           // byte offset in the arena header of the chains' row-block counters
  size_t chain_counter_words = 0;
  size_t header_clear_bytes = 256;        // what a run zeroes at the start of the arena (status word, tickets, chain counters)
  // Staged planning (exact handling of execution-determined extents): `pinned` roots keep the arena offsets an
  // earlier stage gave them; `front_reserve` > 0 puts the group scratch (front_scratch bytes) and the Switch index
  // lists behind the header instead of behind the tensors, so that neither moves between stages.
  std::vector<std::pair<int, size_t>> pinned;
  size_t front_reserve = 0, front_scratch = 0, header_end = 0;
  // a staged plan lays out only the tensors of its own steps: those defined at or before place_until_step and still
  // live at place_from_step (earlier ones are dead, later ones are planned by a later stage, at their true sizes)
  int place_from_step = 0, place_until_step = 1 << 30;
  // [group] run-time symbols (atom ids) whose counts are in the arena header once the group has run: a gate whose
  // kernel also partitions the sample ids, a Switch that partitions them itself, a NonZero
  std::vector<std::vector<int>> rt_syms_after;
  // OPT_GUARD_BANDS: (arena offset of a 256-byte band, tensor it follows or -1 = scratch, -2 = index lists)
  std::vector<std::pair<size_t, int>> guard_bands;
  std::string err;
  // device status word lives at arena offset 0 (first 256 bytes reserved)
  // CUDA graph of the whole launch sequence for one set of buffers (run_plan_graph)
  void* graph_exec = nullptr;             // cudaGraphExec_t
  void* capture_stream = nullptr;         // cudaStream_t the sequence is captured on
  // groups that run beside their predecessor on a second stream (forked before the predecessor's first launch,
  // joined after their own last one): both only read what came before and write their own outputs
  std::vector<char> side_group;           // [group]
  void* side_stream = nullptr;            // cudaStream_t
  void* ev_fork = nullptr;                // cudaEvent_t
  void* ev_join = nullptr;                // cudaEvent_t
  std::vector<const void*> graph_key;     // inputs, outputs, arena the graph was captured with
  Plan() = default;
  Plan(const Plan&) = delete;
  Plan& operator=(const Plan&) = delete;
  ~Plan();                                // exec.cu: releases the graph and the capture stream
};
Status make_plan(const Compiled* c, const Binding* b, Plan* p);
// The launch sequence of run_plan as one CUDA graph: captured (on a stream of the plan's own, so that
// the caller may pass the legacy default stream) the first time and whenever an input, output or arena
// pointer differs from the captured ones, then replayed on `stream`.  info[3] = 1 if this call captured.
Status run_plan_graph(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream,
                      int64_t* info);
Status build_launches(Plan* p);   // exec.cu
Status detect_chains(Plan* p);    // exec.cu: fills Plan::chains / chain_of from the resolved views
// step_lo..step_hi: only these groups (positions in execution order) are enqueued (all by default); the arena header
// is cleared only by a run that starts at group 0.
Status run_plan(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream,
                int64_t* info, int step_lo = 0, int step_hi = 1 << 30);

// Exact handling of execution-determined extents: see exec.cu.  `bounded` is the ordinary plan of b0 (its scratch
// sizes fix the layout in front of the tensors); the arena must hold at least bounded->arena_bytes.
Status run_exact(const Compiled* c, const Binding* b0, const Plan* bounded, const void* const* inputs, void* const* outputs, void* arena,
                 size_t arena_bytes, void* stream, int64_t* info, std::string* err);

// Guard bands (OPT_GUARD_BANDS): fill the arena behind the header with 0xFF bytes; count the bands a run damaged.
Status poison_arena(const Plan* p, void* arena, size_t arena_bytes, void* stream);
Status check_guards(const Plan* p, void* arena, void* stream, int* n_bad, int* first_tensor);

// Same as run_plan, with CUDA events around every launch; synchronises the stream and returns the
// device time per group (ms).
// reps > 1: every launch is issued `reps` times back to back between its two events and the time divided by reps
// (the kernel's duration without the idle gap between an event and a lone launch); only meaningful where a
// launch may be repeated without changing its inputs.
Status run_plan_timed(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream,
                      float* group_ms, int n_groups, int reps = 1);

}  // namespace sod2
