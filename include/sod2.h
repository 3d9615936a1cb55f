/* sod2.h — C ABI of the B200-native SoD^2 hot path.
 *
 * The library executes the fused operator groups that Rank-and-Dimension Propagation (RDP) makes
 * possible on dynamic DNNs.  The calls follow the staging the paper describes: static analysis before
 * deployment (Section 4.1-4.3: operator classification, RDP = Algorithm 1, fusion, partition at
 * execution-determined operators), then, per input, evaluation of the shape expressions and the
 * memory allocation plan, made once the input has fixed every tensor size (Section 4.4.1), then
 * inference.
 *
 * Conventions
 *  - Every call returns a sod2_status, never throws, never aborts, never prints.  Out-parameters
 *    are untouched on error.  sod2_last_error(handle) gives a message for the last failure.
 *  - Handles are owned by the library and freed by the matching *_destroy.
 *  - ALL DEVICE MEMORY IS OWNED BY THE CALLER: inputs, outputs, constants, the prepack workspace and
 *    the arena.  The library never allocates or frees device memory.
 *  - Batches: a graph is written for ONE request; sod2_bind_dims binds n_requests at once.  Every
 *    input / output / arena tensor holds the requests' instances back to back in request order
 *    (instance sizes rounded up to 16 bytes), e.g. x:[1,L,768] for 8 requests is one packed
 *    [sum L, 768] buffer.  No padding to a maximum length exists anywhere.
 *  - Pointers named dev_* / inputs / outputs / arena / workspace are DEVICE pointers; all others are
 *    host pointers.  cuda_stream is a cudaStream_t passed as void*.
 *  - One thread per handle.  Same inputs => bit-identical outputs (Section 4: deterministic).
 */
#ifndef SOD2_H_
#define SOD2_H_
#include <stddef.h>
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

typedef struct sod2_graph sod2_graph;
typedef struct sod2_binding sod2_binding;
typedef struct sod2_plan_s sod2_plan_t;

typedef enum {
  SOD2_OK = 0, SOD2_E_INVALID_ARG, SOD2_E_PARSE, SOD2_E_UNSUPPORTED_OP, SOD2_E_RANK_MISMATCH,
  SOD2_E_NOT_CONVERGED, SOD2_E_UNBOUND_SYMBOL, SOD2_E_BAD_DIM, SOD2_E_SHAPE_CONFLICT,
  SOD2_E_ARENA_TOO_SMALL, SOD2_E_MISALIGNED, SOD2_E_CUDA, SOD2_E_TIMEOUT, SOD2_E_INTERNAL
} sod2_status;

/* option bits for sod2_graph_create */
#define SOD2_OPT_NO_FUSION 1u /* every operator is its own group */
#define SOD2_OPT_NO_REUSE  2u /* every arena tensor keeps its own slot: intermediates stay readable */
#define SOD2_OPT_COPY_REGROUP 16u /* Switch / Combine always copy whole samples (no index-indirect convolutions) */
#define SOD2_OPT_LEGACY_ATTENTION 8u /* attention groups run the mma.sync kernel even where the tcgen05 kernel applies */
#define SOD2_OPT_MULTI_VERSION 64u /* fuse elementwise chains across broadcasts RDP cannot resolve: 2^d fused versions (Section 4.2), the version (a stride table) chosen at bind time */
#define SOD2_OPT_NO_SEP 32u /* groups run in their default topological order: no static execution planning (Section 4.3) */
#define SOD2_OPT_LN_FOLD 128u /* a LayerNorm between bf16 GEMMs is folded into its neighbours (Section 4.2: fusion removes the materialised intermediate): the producing GEMM writes per-row statistics, the consuming GEMMs read the raw rows and normalise in their epilogues, the normalised tensor is never stored.  Opt-in: measured slower on the encoder workloads, where the LayerNorm kernel runs beside the next GEMM's pipeline fill */
#define SOD2_OPT_GUARD_BANDS 512u /* debugging aid: every arena tensor gets a slot of its own (a band another tensor may cover at another time proves nothing) with 256 bytes behind it, also behind the scratch regions (sod2_plan_poison_arena / sod2_plan_check_guards) */
#define SOD2_OPT_GEMM_PAIR 1024u /* bf16 GEMMs on CTA pairs: two CTAs of a cluster share a 256 x N tile, each loading its own rows and half of the weight tile (tcgen05.mma.cta_group::2), chosen per bound shape where the estimated makespan is shorter (Section 4.4.2: one more code version).  Opt-in: results equal the single-CTA kernel's; measured 0.5 - 1.5 us slower per kernel at a few thousand rows, where the main loop does not wait for operands and the cluster launch costs more than the saved loads */
#define SOD2_OPT_GEMM_CHAIN 256u /* consecutive GEMM groups that depend on each other row block by row block run as one persistent kernel with per-row-block dependency counters in the arena header (their operands stay live over the whole chain).  Opt-in: measured slower than one launch per GEMM at a few thousand rows */
#define SOD2_OPT_SPLITK_LN 4u /* bf16 GEMM (+bias, +residual) -> LayerNorm as one group: split-K GEMM into fp32 slabs + finishing kernel */

/* Parse the graph text (host, ir_len bytes), classify every operator (Table 2), run RDP
 * (Algorithm 1) to a fixpoint, form fused groups (Section 4.2) and partition at
 * execution-determined operators (Section 4.3).  Pure host work, no CUDA call. */
sod2_status sod2_graph_create(const char* ir_text, size_t ir_len, uint32_t opt_flags, sod2_graph** out);
void sod2_graph_destroy(sod2_graph* g);

/* Attach caller-owned device memory holding a float constant (weights: the constant inputs of the
 * computational graph, Section 3) in the layout the graph
 * declares (row-major, graph dtype).  The memory must outlive every run. */
sod2_status sod2_graph_set_const(sod2_graph* g, const char* name, const void* dev_ptr, size_t bytes);

/* GEMM weights are re-laid K-major for the tensor-core kernel.  Query the workspace size, then
 * prepack once into caller-owned device memory (256-byte aligned); the copies are enqueued on
 * cuda_stream and must complete before the first run. */
sod2_status sod2_graph_prepack_bytes(const sod2_graph* g, size_t* bytes);
sod2_status sod2_graph_prepack(sod2_graph* g, void* dev_workspace, size_t bytes, void* cuda_stream);

/* H0: bind symbol values for n_requests requests (Section 4.1: the symbolic constants of the RDP
 * lattice get their values once an input arrives; Section 4.4.1: all sizes are then known).  values is [n_requests][n_syms] row-major (host).
 * Evaluates every shape expression of every tensor for every request and checks the bind-time
 * assertions RDP recorded.  Errors: unknown / unbound symbol, value outside the declared range,
 * shape conflict. */
sod2_status sod2_bind_dims(sod2_graph* g, int n_requests, int n_syms, const char* const* sym_names,
                           const int64_t* values, sod2_binding** out);
void sod2_binding_destroy(sod2_binding* b);

/* H1+H2: arena memory plan (Section 4.4.1, peak-first greedy over one linear arena), kernel-variant
 * choice by shape class (Section 4.4.2) and launch parameters.  arena_bytes = size the caller must
 * provide to sod2_run.  The binding must outlive the plan. */
sod2_status sod2_plan(sod2_graph* g, const sod2_binding* b, sod2_plan_t** out, size_t* arena_bytes);
void sod2_plan_destroy(sod2_plan_t* p);

/* Plan cache.  Planning happens at execution time, when the sizes are known (Section 4.4.1); a request
 * mix whose bound symbol tuple has been seen before needs no new plan.  sod2_graph_set_plan_cache sets
 * the number of (binding, plan) pairs the graph keeps, least recently used first out (0, the default,
 * disables and empties the cache).  sod2_plan_cached = sod2_bind_dims + sod2_plan through the cache:
 * *hit = 1 if the pair was found.  The handles it returns are BORROWED: they belong to the graph and
 * stay valid until the entry is evicted by later misses, the capacity is lowered or the graph is
 * destroyed; sod2_binding_destroy / sod2_plan_destroy ignore them.  A plan does not depend on the
 * addresses it ran with, so a cached plan may be run with any inputs, outputs and arena. */
sod2_status sod2_graph_set_plan_cache(sod2_graph* g, int capacity);
sod2_status sod2_plan_cached(sod2_graph* g, int n_requests, int n_syms, const char* const* sym_names,
                             const int64_t* values, sod2_binding** binding_out, sod2_plan_t** plan_out,
                             size_t* arena_bytes, int* hit);

typedef struct {
  int64_t host_enqueue_ns; /* host time spent inside sod2_run */
  int64_t gpu_launches;    /* kernels enqueued */
  int64_t reserved[6];
} sod2_run_info;

/* Enqueue one inference (all requests of the binding) on cuda_stream: the fused groups (Section 4.2) of
 * each sub-graph of the partition at execution-determined operators (Section 4.3), in planned order, in
 * the arena laid out by sod2_plan (Section 4.4.1), each group by the kernel version chosen for its bound
 * shapes (Section 4.4.2).  inputs[i] / outputs[j] are
 * device pointers in graph declaration order, packed per request as described above; outputs whose
 * shape is execution-determined must be sized for the static upper bound (sod2_binding_shape reports
 * it) and their true shape is read with sod2_run_output_shape after the stream has been synchronised.
 * arena: >= arena_bytes, 256-byte aligned (SOD2_E_ARENA_TOO_SMALL / SOD2_E_MISALIGNED).  Asynchronous.
 * Device-side failures (a bounded wait that ran out) are reported by sod2_plan_device_status. */
sod2_status sod2_run(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena,
                     size_t arena_bytes, void* cuda_stream, sod2_run_info* info);

/* The same inference as one CUDA graph.  The plan's launch sequence is captured (on a stream owned by the
 * plan, so cuda_stream may be the legacy default stream) the first time, and again whenever an input,
 * output or arena pointer differs from the captured ones; otherwise the instantiated graph is replayed on
 * cuda_stream.  Same kernels, same results; the host enqueues one graph launch instead of one launch per
 * kernel and the device-side gaps between dependent kernels shrink (cfg 3: 0.73 -> 0.67 ms).  For serving
 * loops that keep their buffers; a call that has to capture costs about a millisecond of host time.
 * info->reserved[1] = 1 if this call captured.  The graph is released with the plan. */
sod2_status sod2_run_graph(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena,
                           size_t arena_bytes, void* cuda_stream, sod2_run_info* info);

/* The same inference with EXACT handling of execution-determined extents, the staging the paper describes
 * (Section 3: the output shape of such an operator is known only once it has run; Section 4.3: the graph is
 * partitioned at these operators; Section 4.4.1: memory is planned when the sizes are known).  p is the ordinary
 * (bounded) plan of the binding: sod2_run keeps every count on the device and plans such tensors at their static
 * upper bound, one uninterrupted launch sequence.  Here the sub-graphs of the partition run one after another; after
 * each sub-graph that holds a Switch or NonZero the counts are copied to the host (the call SYNCHRONISES cuda_stream
 * there), the run-time symbols are bound to them and the remaining sub-graphs are planned again at their true sizes:
 * tensors that already exist keep their arena offsets, the others are laid out around them; group scratch and the
 * Switch index lists sit at fixed offsets behind the arena header.  Same kernels, same results.  arena as for
 * sod2_run (>= the bounded plan's arena_bytes).  info->reserved[2] = stages planned, reserved[3] = largest arena
 * extent (bytes) any stage laid out (a stage places only the tensors of its own sub-graphs); reserved[4] = host nanoseconds spent binding and planning the stages.
 * Errors as sod2_run, plus SOD2_E_ARENA_TOO_SMALL if a stage planned around the tensors in place does not fit. */
sod2_status sod2_run_exact(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena,
                           size_t arena_bytes, void* cuda_stream, sod2_run_info* info);

/* Debugging aids for graphs created with SOD2_OPT_GUARD_BANDS (they stand in for a memory checker: every kernel of
 * the library takes its bounds from the plan, Section 4.4.1, so a store past the end of a planned tensor is a
 * planning or kernel defect).  sod2_plan_poison_arena fills the arena behind its header with 0xFF bytes (NaN in bf16
 * and fp32: a read of memory that nothing wrote shows up in the results); call it before sod2_run.
 * sod2_plan_check_guards, after the run, counts the 256-byte bands behind tensors and scratch regions that no longer
 * hold those bytes (*n_damaged) and names the tensor behind which the lowest damaged band lies (first_name, host
 * buffer, may be NULL).  It overwrites header bytes 16..127 and synchronises cuda_stream.  Errors:
 * SOD2_E_INVALID_ARG (graph without the option), SOD2_E_ARENA_TOO_SMALL, SOD2_E_CUDA. */
sod2_status sod2_plan_poison_arena(sod2_plan_t* p, void* arena, size_t arena_bytes, void* cuda_stream);
sod2_status sod2_plan_check_guards(sod2_plan_t* p, void* arena, void* cuda_stream, int* n_damaged, char* first_name,
                                   size_t first_name_len);

/* Measurement aid: the same inference with CUDA events recorded on cuda_stream around every launch.
 * Synchronises the stream and returns the device time of each fused group in group_ms[n_groups]
 * (host array, milliseconds; n_groups must equal sod2_graph_num_groups).  A launch that runs several
 * groups (a chain of GEMMs) is divided among them in proportion to their algorithmic flops. */
sod2_status sod2_run_timed(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena,
                           size_t arena_bytes, void* cuda_stream, float* group_ms, int n_groups);

/* The same with every launch issued `reps` times back to back between its two events, the time divided by
 * reps: a kernel's duration as it is inside a busy stream, without the idle gap that follows an event when
 * a lone launch has to travel from the host.  The repeated launches recompute the same values (results of
 * groups that update a tensor in place, the gated convolutions, are not meaningful afterwards): a measuring
 * aid for the encoder workloads. */
sod2_status sod2_run_timed_repeat(sod2_plan_t* p, const void* const* inputs, void* const* outputs, void* arena,
                                  size_t arena_bytes, void* cuda_stream, int reps, float* group_ms, int n_groups);

/* Reads the device status word written by the last run (synchronises the stream).
 * SOD2_OK, or SOD2_E_TIMEOUT if a kernel gave up on a bounded wait. */
sod2_status sod2_plan_device_status(sod2_plan_t* p, const void* arena, void* cuda_stream);

/* ---- introspection (used by the tests that check the RDP shape expressions) ---- */
/* rank: -1 undef, -2 nac.  dim_kind[i]: 0 undef, 1 known constant, 2 symbolic constant,
 * 3 operation-inferred expression, 4 nac (execution determined).  expr_buf receives the shape as
 * "[e0,e1,...]" in canonical form.  dim_kind may be NULL; it must hold `rank` ints otherwise. */
sod2_status sod2_graph_tensor_info(const sod2_graph* g, const char* tensor, int* rank, int* dim_kind,
                                   char* expr_buf, size_t expr_buf_len);
/* Element type of a tensor: 0 f32, 1 bf16, 2 i64, 3 bool (1 byte). */
sod2_status sod2_graph_tensor_dtype(const sod2_graph* g, const char* tensor, int* dtype);
/* Value-map entry of a small integer tensor as "[e0,...]", "undef" or "nac". */
sod2_status sod2_graph_tensor_value(const sod2_graph* g, const char* tensor, char* buf, size_t buf_len);
int sod2_graph_num_ops(const sod2_graph* g);
/* dyn_class / eff_class: 0 ISDO, 1 ISDOS, 2 ISVDOS, 3 EDO (Table 2; eff_class after constant
 * propagation).  group_id: -1 for operators evaluated by RDP itself or pure views. */
sod2_status sod2_graph_op_info(const sod2_graph* g, int op, char* op_type, size_t op_type_len, int* dyn_class,
                               int* eff_class, int* group_id, int* subgraph_id);
int sod2_graph_num_groups(const sod2_graph* g);
/* kind_buf: group kernel kind name; versions: fused code versions needed (1 when RDP resolved every
 * broadcast); n_ops: operators fused into the group. */
sod2_status sod2_graph_group_info(const sod2_graph* g, int group, char* kind_buf, size_t kind_len, int* n_ops,
                                  int* versions, int* subgraph_id);
int sod2_graph_num_subgraphs(const sod2_graph* g);
int sod2_graph_rdp_sweeps(const sod2_graph* g);
/* Static execution planning (Section 4.3): the order of the fused groups inside each sub-graph of the
 * nac partition is the one of least peak live intermediate bytes, found by a search over all
 * topological orders with tensor sizes taken at the upper bounds of the declared symbol ranges
 * (lower bounds break ties).  out[0], out[1]: peak live bytes of the default order at the upper and
 * lower corner; out[2], out[3]: the same for the planned order; out[4]: sets of finished groups the
 * search visited; out[5], out[6], out[7]: sub-graphs searched, reordered, abandoned (state budget
 * exceeded: default order kept); out[8]: 1 if some tensor size has no static bound (nothing searched).
 * `out` is host memory for 9 values.  All zero under SOD2_OPT_NO_SEP. */
sod2_status sod2_graph_order_info(const sod2_graph* g, int64_t* out);
/* Classification of an operator name alone (Table 2). Returns SOD2_E_UNSUPPORTED_OP if unknown. */
sod2_status sod2_classify(const char* op_type, int* dyn_class);
/* Re-run RDP visiting the operators in the given order (a permutation of 0..num_ops-1); used to
 * check that the fixpoint does not depend on the order. Must be called before any bind. */
sod2_status sod2_graph_reanalyse(sod2_graph* g, const int* order, int n);

sod2_status sod2_binding_shape(const sod2_binding* b, int request, const char* tensor, int64_t* dims, int* rank);
/* Arena slot of an inter-group tensor: byte offset, byte size (all requests), defining and last-using step. */
sod2_status sod2_plan_slot(const sod2_plan_t* p, const char* tensor, size_t* offset, size_t* bytes, int* def_step,
                           int* last_use_step);
/* Byte offset of one request's instance inside a packed tensor buffer. */
sod2_status sod2_plan_instance_offset(const sod2_plan_t* p, const char* tensor, int request, size_t* offset);
/* Element strides of one request's instance of a tensor in its buffer (views and channels-last
 * storage are not contiguous in the logical dim order). strides must hold `rank` entries. */
sod2_status sod2_plan_tensor_strides(const sod2_plan_t* p, const char* tensor, int request, int64_t* strides, int* rank);
/* arena_bytes, peak live bytes, sum of all inter-group tensor bytes (what no-reuse allocation takes). */
sod2_status sod2_plan_memory(const sod2_plan_t* p, size_t* arena_bytes, size_t* peak_live_bytes, size_t* sum_bytes);
/* Algorithmic cost of one fused group for the bound shapes: flops of its contraction (0 for
 * HBM-bound groups) and bytes = every external input and output once, constants once, nothing for
 * tensors that stay inside the group. */
sod2_status sod2_plan_group_cost(const sod2_plan_t* p, int group, double* flops, double* bytes);
/* *on_side = 1 if the group's kernels run on the plan's second stream beside the previous group (Section 4.3 orders
 * the groups; two consecutive groups overlap only where neither reads what the other writes AND both read the same
 * tensor, so that the memory plan, which knows liveness by step, cannot hand one of them a slot the other still
 * reads), else 0. */
sod2_status sod2_plan_group_on_side_stream(const sod2_plan_t* p, int group, int* on_side);
/* True shape of an output after a run (execution-determined extents are read back from the device;
 * synchronises cuda_stream). */
sod2_status sod2_run_output_shape(sod2_plan_t* p, const void* arena, void* cuda_stream, int request, int output,
                                  int64_t* dims, int* rank);

/* NonZero without any allocation: for callers that cannot call cudaMalloc (code inside a stream
 * capture or a serving loop where an allocation would synchronise the device, plug-ins whose host
 * framework owns all device memory and hands out only input and output buffers, processes under a
 * fixed memory budget) and therefore cannot provide an arena either.  The paper has no counterpart
 * of this call; it is a packaging variant of the NonZero compaction above.
 *   dev_x     device, [dims...] row-major, dtype 0 = f32, 1 = bf16; rank 1..4; dims on the host
 *   dev_out   device, int64 [rank, nnz] with row pitch nnz; must hold rank * numel entries
 *   dev_count device, one int64: receives nnz
 * The scratch (per-block counters) is a fixed array inside the library's device image: inputs of
 * more than SOD2_NONZERO_STATIC_MAX_ELEMS elements are rejected with SOD2_E_BAD_DIM; every GPU that
 * loads the library holds the array (about 65 KB) until the process exits; all calls share it, so
 * calls that overlap on the GPU (two streams, two threads) race; it keeps the previous call's
 * contents, which is harmless because every call overwrites each counter before reading it.  The
 * first call on a device looks up the array's address and should be made outside any stream
 * capture.  The device that holds dev_x must be the current device and own cuda_stream.  Calls no
 * cudaMalloc / cudaFree or allocating routine.  Asynchronous on cuda_stream.
 * Errors: SOD2_E_INVALID_ARG, SOD2_E_RANK_MISMATCH, SOD2_E_BAD_DIM, SOD2_E_CUDA; message through
 * sod2_last_error(NULL). */
#define SOD2_NONZERO_STATIC_MAX_ELEMS 16777216LL
sod2_status sod2_nonzero_static(const void* dev_x, int dtype, int rank, const int64_t* dims, int64_t* dev_out,
                                int64_t* dev_count, void* cuda_stream);

/* Launches one kernel that does nothing (one thread, no arguments) on cuda_stream.  A measuring aid:
 * the smallest fused groups (a few thousand elements per request) take about as long as this launch,
 * so their time is reported as a multiple of it rather than as a fraction of a roofline.
 * Asynchronous.  Errors: SOD2_E_CUDA; message through sod2_last_error(NULL). */
sod2_status sod2_launch_empty(void* cuda_stream);

/* Self-test of the bounded waits (Section 4: deterministic sequence of operations; a wait that cannot complete
 * must end, not hang the device).  Launches one small kernel on cuda_stream that waits, with the library's
 * bounded wait and a limit of 4096 polls, on a barrier nothing arrives on; the wait runs out, the kernel writes 1
 * to the device word dev_status_word (the first word of an arena: what sod2_plan_device_status reads) and returns by
 * itself.  Nothing traps and nothing waits without a limit.  Asynchronous.  Errors: SOD2_E_INVALID_ARG,
 * SOD2_E_CUDA; message through sod2_last_error(NULL). */
sod2_status sod2_selftest_bounded_wait(void* dev_status_word, void* cuda_stream);

/* Measurement of the tensor pipe's issue rate (no counterpart in the paper: it records the machine facts behind the
 * multi-version kernels of Section 4.4.2 and lets a test pin them).  On `clusters` pairs of SMs (1..74), one thread
 * per CTA (pair = 0: tcgen05.mma.cta_group::1, 128 x n_cols x 16, both CTAs of every cluster at once) or one per CTA
 * pair (pair = 1: cta_group::2, 256 x n_cols x 16) issues `iters` bf16 MMAs on fixed shared-memory operands, in
 * stages of `per_stage` instructions.  handshake: 0 = MMAs only, 1 = a tcgen05.commit after every stage, 2 = the
 * full / empty barrier handshake of the GEMM main loops after every stage (all waits satisfied at once).
 * *cycles_per_mma (host) = SM cycles of the first issuing thread / iters.  n_cols in {64, 128, 256}; per_stage in
 * 1..64 and dividing iters; iters <= 65536.  Allocates and frees one small device buffer; synchronises cuda_stream.
 * Every wait in the kernel is bounded.  Errors: SOD2_E_INVALID_ARG, SOD2_E_CUDA, SOD2_E_TIMEOUT (a wait ran out);
 * message through sod2_last_error(NULL). */
sod2_status sod2_selftest_mma_rate(int pair, int n_cols, int per_stage, int handshake, int iters, int clusters,
                                   void* cuda_stream, double* cycles_per_mma);

/* handle may be a graph, binding or plan; returns "" if there was no error. */
const char* sod2_last_error(const void* any_handle);

#ifdef __cplusplus
}
#endif
#endif /* SOD2_H_ */
