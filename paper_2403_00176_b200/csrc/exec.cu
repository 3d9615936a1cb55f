// Launch plan (variant choice, tensor maps, kernel parameters) and the executor that enqueues the
// fused groups on the caller's stream.  All device memory belongs to the caller; this file never
// allocates device memory.
#include <chrono>
#include <cmath>
#include <cstring>
#include <functional>
#include <map>
#include <set>

#include "attention.cuh"
#include "attention_tcgen05.cuh"
#include "conv_tcgen05.cuh"
#include "conv3x3_tcgen05.cuh"
#include "conv_stem_tcgen05.cuh"
#include "engine.h"
#include "gemm_tcgen05.cuh"
#include "gemm_chain_tcgen05.cuh"
#include "gemm_pair_tcgen05.cuh"
#include "kernels_compact.cuh"
#include "kernels_rows.cuh"
#include "kernels_unfused.cuh"
#include "tmap.h"

namespace sod2 {

struct RunCtx {
  const void* const* inputs;
  void* const* outputs;
  char* arena;
  char* packed;
  cudaStream_t stream;
  const Plan* plan;
  char* resolve(const Ptr& p) const {
    switch (p.where) {
      case RootBuf::INPUT: return const_cast<char*>(static_cast<const char*>(inputs[p.index])) + p.off;
      case RootBuf::OUTPUT: return static_cast<char*>(outputs[p.index]) + p.off;
      case RootBuf::CONST: return const_cast<char*>(static_cast<const char*>(plan->c->g.tensors[p.index].dev_ptr)) + p.off;
      case RootBuf::ARENA: return arena + p.off;
      case 5: return packed + p.off;
      default: return nullptr;
    }
  }
};

struct Launch {
  int group = -1;
  int n_kernels = 1;
  std::function<cudaError_t(const RunCtx&)> fn;
  // a launch that runs several groups (a GEMM chain): (group, share of the launch's time by algorithmic flops)
  std::vector<std::pair<int, double>> share;
};

namespace {

// Launch with programmatic dependent launch allowed (see ptx::pdl_wait): only for kernels that call
// pdl_wait() in every thread.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// The same with a thread-block cluster of two CTAs along x (the CTA-pair GEMM).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_pair(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

int64_t numel(const DimVec& d) { int64_t n = 1; for (auto v : d) n *= v; return n; }

// The RGB stem has a kernel of its own (conv_stem_tcgen05.cuh): 7x7, stride 2, padding 3, 3 -> 64 channels,
// bias, no or ReLU activation.  Decided per graph, so that the weights are prepacked in its K order.
bool is_fused_stem(const Compiled& c, const Group& G) {
  if (G.kind != GKind::CONV || G.w < 0 || G.res >= 0 || G.act2 || G.has_ln || (G.act != 0 && G.act != 2)) return false;
  const Tensor& W = c.g.tensors[G.w];
  if (W.dtype != DType::BF16 || W.S.rank != 4) return false;
  for (int i = 0; i < 4; ++i) if (!W.S.dims[i].known() || !W.S.dims[i].e.is_const()) return false;
  return W.S.dims[0].e.const_value() == 64 && W.S.dims[1].e.const_value() == 3 && W.S.dims[2].e.const_value() == 7 &&
         W.S.dims[3].e.const_value() == 7 && G.stride == 2 && G.pad == 3;
}

// One instantiation of the tcgen05 GEMM: sets its shared-memory limit once and launches it with programmatic
// dependent launch.
template <int BN, int KCH, int ST, int ACT, bool RES, int LN, bool EMIT>
cudaError_t launch_gemm_variant(dim3 grid, cudaStream_t st, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                                const CUtensorMap& tr, int M, int N, int K, const k::GemmEpilogue& ep) {
  constexpr int smem = k::GemmSmem<BN, KCH, ST>::TOTAL;
  static bool once = (cudaFuncSetAttribute(k::gemm_bf16_tcgen05<BN, KCH, ST, ACT, false, RES, LN, EMIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);
  (void)once;
  return launch_pdl(k::gemm_bf16_tcgen05<BN, KCH, ST, ACT, false, RES, LN, EMIT>, grid, dim3(k::GEMM_THREADS), smem, st, ta, tb, to, tr, M, N, K, ep);
}
// Epilogue versions of one tile version: plain (activation x residual), normalised A operand (LN = 1, any
// activation), normalised residual (LN = 2, tiles up to 128 wide), each of the residual forms with or without
// row statistics of the output (EMIT).
template <int BN, int KCH, int ST>
cudaError_t gemm_dispatch(int act, bool res, int ln, bool emit, dim3 grid, cudaStream_t st, const CUtensorMap& ta, const CUtensorMap& tb,
                          const CUtensorMap& to, const CUtensorMap& tr, int M, int N, int K, const k::GemmEpilogue& ep) {
#define SOD2_GV(ACT_, RES_, LN_, EMIT_) return launch_gemm_variant<BN, KCH, ST, ACT_, RES_, LN_, EMIT_>(grid, st, ta, tb, to, tr, M, N, K, ep)
  if (ln == 0 && !emit) {
    switch (act * 2 + (res ? 1 : 0)) {
      case 0: SOD2_GV(0, false, 0, false);
      case 1: SOD2_GV(0, true, 0, false);
      case 2: SOD2_GV(1, false, 0, false);
      case 3: SOD2_GV(1, true, 0, false);
      case 4: SOD2_GV(2, false, 0, false);
      default: SOD2_GV(2, true, 0, false);
    }
  }
  if (ln == 1 && !res && !emit) {
    switch (act) {
      case 0: SOD2_GV(0, false, 1, false);
      case 1: SOD2_GV(1, false, 1, false);
      default: SOD2_GV(2, false, 1, false);
    }
  }
  if (act != 0) return cudaErrorInvalidValue;
  if (ln == 2 && res) {
    if constexpr (BN <= 128) {
      if (emit) SOD2_GV(0, true, 2, true);
      SOD2_GV(0, true, 2, false);
    }
    return cudaErrorInvalidValue;
  }
  if (ln == 0 && emit) {
    if (res) SOD2_GV(0, true, 0, true);
    SOD2_GV(0, false, 0, true);
  }
#undef SOD2_GV
  return cudaErrorInvalidValue;
}

template <int BN, int KCH, int ST, int ACT, bool RES>
cudaError_t launch_gemm_pair_variant(dim3 grid, cudaStream_t st, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                                     const CUtensorMap& tr, int M, int N, int K, const k::GemmEpilogue& ep) {
  constexpr int smem = k::GemmPairSmem<BN, KCH, ST>::TOTAL;
  static bool once = (cudaFuncSetAttribute(k::gemm_pair_bf16_tcgen05<BN, KCH, ST, ACT, RES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);
  (void)once;
  return launch_pdl_pair(k::gemm_pair_bf16_tcgen05<BN, KCH, ST, ACT, RES>, grid, dim3(k::GEMM_THREADS), smem, st, ta, tb, to, tr, M, N, K, ep);
}
template <int BN, int KCH, int ST>
cudaError_t gemm_pair_dispatch(int act, bool res, dim3 grid, cudaStream_t st, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                               const CUtensorMap& tr, int M, int N, int K, const k::GemmEpilogue& ep) {
  switch (act * 2 + (res ? 1 : 0)) {
    case 0: return launch_gemm_pair_variant<BN, KCH, ST, 0, false>(grid, st, ta, tb, to, tr, M, N, K, ep);
    case 1: return launch_gemm_pair_variant<BN, KCH, ST, 0, true>(grid, st, ta, tb, to, tr, M, N, K, ep);
    case 2: return launch_gemm_pair_variant<BN, KCH, ST, 1, false>(grid, st, ta, tb, to, tr, M, N, K, ep);
    case 3: return launch_gemm_pair_variant<BN, KCH, ST, 1, true>(grid, st, ta, tb, to, tr, M, N, K, ep);
    case 4: return launch_gemm_pair_variant<BN, KCH, ST, 2, false>(grid, st, ta, tb, to, tr, M, N, K, ep);
    default: return launch_gemm_pair_variant<BN, KCH, ST, 2, true>(grid, st, ta, tb, to, tr, M, N, K, ep);
  }
}

struct Builder {
  Plan& p;
  const Compiled& c;
  const Graph& g;
  size_t scratch_need = 0;
  explicit Builder(Plan& pp) : p(pp), c(*pp.c), g(pp.c->g) {}

  Status fail(Status s, const std::string& m) { p.err = m; return s; }

  Ptr ptr_of(int t, int r, int64_t extra_elems = 0) const {
    const View& v = p.views[t][r];
    const int root = p.root_of[t];
    const RootBuf& R = p.roots[root];
    Ptr q;
    q.where = R.where;
    q.index = (R.where == RootBuf::CONST) ? root : R.io_index;
    q.off = p.inst_off[root][r] + (v.offset + extra_elems) * dtype_size(g.tensors[t].dtype);
    if (R.where == RootBuf::ARENA) q.off += static_cast<int64_t>(R.arena_off);
    return q;
  }
  static bool same_base(const Ptr& a, const Ptr& b) { return a.where == b.where && a.index == b.index; }

  // collapse a view to [rows, cols] with unit column stride; returns row pitch in elements
  bool as_matrix(const View& v, int64_t* rows, int64_t* cols, int64_t* ld) const {
    if (v.dims.empty()) return false;
    *cols = v.dims.back();
    *rows = numel(v.dims) / std::max<int64_t>(*cols, 1);
    if (v.strides.back() != 1 && *cols != 1) return false;
    // all leading dims must step uniformly
    int64_t pitch = -1, run = 1;
    for (int i = static_cast<int>(v.dims.size()) - 2; i >= 0; --i) {
      if (v.dims[i] == 1) continue;
      if (pitch < 0) { pitch = v.strides[i]; run = v.dims[i]; }
      else { if (v.strides[i] != pitch * run) return false; run *= v.dims[i]; }
    }
    *ld = pitch < 0 ? *cols : pitch;
    return true;
  }

  // rows of consecutive requests that form one contiguous matrix are merged into one launch
  struct Seg { int r0, r1; int64_t rows; };
  std::vector<int64_t> row_count_;
  Status row_segments(const std::vector<int>& tensors, int64_t* cols_out, std::vector<int64_t>* lds, std::vector<Seg>* segs) {
    int nt = static_cast<int>(tensors.size());
    lds->assign(nt, 0);
    row_count_.resize(p.n_req);   // rows of the first tensor, per request (the others must agree)
    for (int i = 0; i < nt; ++i) {
      auto views = p.views[tensors[i]];
      for (int r = 0; r < p.n_req; ++r) {
        int64_t rw, cl, ld;
        if (!as_matrix(views[r], &rw, &cl, &ld)) return fail(E_UNSUPPORTED_OP, "operand " + g.tensors[tensors[i]].name + " is not a row-major matrix view");
        if (r == 0) (*lds)[i] = ld;
        else if (ld != (*lds)[i] && rw > 1) return fail(E_UNSUPPORTED_OP, "row pitch differs between requests");
        if (i == 0) { row_count_[r] = rw; cols_out[0] = cl; }
        if (rw != row_count_[r]) return fail(E_SHAPE_CONFLICT, "row counts differ inside a group");
      }
    }
    segs->clear();
    for (int r = 0; r < p.n_req; ++r) {
      bool merge = !segs->empty();
      for (int i = 0; i < nt && merge; ++i) {
        Ptr a = ptr_of(tensors[i], segs->back().r0), b = ptr_of(tensors[i], r);
        int esz = dtype_size(g.tensors[tensors[i]].dtype);
        if (!same_base(a, b) || b.off != a.off + segs->back().rows * (*lds)[i] * esz) merge = false;
      }
      if (merge) { segs->back().r1 = r + 1; segs->back().rows += row_count_[r]; }
      else segs->push_back({r, r + 1, row_count_[r]});
    }
    return OK;
  }

  void add(int gi, int nk, std::function<cudaError_t(const RunCtx&)> fn) {
    auto L = std::make_shared<Launch>();
    L->group = gi;
    L->n_kernels = nk;
    L->fn = std::move(fn);
    p.gpu_launches += nk;
    p.launches.push_back(L);
  }

  // ------------------------------------------------------------------------------ GEMM
  Status build_gemm(int gi, const Group& G) {
    const Tensor& W = g.tensors[G.w];
    const int64_t K = W.S.dims[0].e.const_value(), N = W.S.dims[1].e.const_value();
    std::vector<int> ts = {G.a, G.out};
    if (G.res >= 0) ts.push_back(G.res);
    int64_t cols;
    std::vector<int64_t> lds;
    std::vector<Seg> segs;
    Status s = row_segments(ts, &cols, &lds, &segs);
    if (s != OK) return s;
    if (cols != K) return fail(E_SHAPE_CONFLICT, "GEMM inner dims differ");
    const bool f32 = g.tensors[G.a].dtype == DType::F32;
    if (f32) {
      if (K > 128 || N > 128 || N % 32) return fail(E_UNSUPPORTED_OP, "fp32 fused group supports K, N <= 128, N % 32 == 0");
      if (lds[0] != K || lds[1] != N || (G.res >= 0 && lds[2] != N)) return fail(E_UNSUPPORTED_OP, "fp32 fused group needs dense rows");
      for (auto& sg : segs) {
        if (sg.rows == 0) continue;
        Ptr pa = ptr_of(G.a, sg.r0), po = ptr_of(G.out, sg.r0), pr = G.res >= 0 ? ptr_of(G.res, sg.r0) : Ptr();
        Ptr pw = ptr_of(G.w, 0), pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr(), pg = G.has_ln ? ptr_of(G.gamma, 0) : Ptr(), pbe = G.has_ln ? ptr_of(G.beta, 0) : Ptr();
        k::MlpLnParams mp{};
        mp.M = static_cast<int>(sg.rows); mp.K = static_cast<int>(K); mp.N = static_cast<int>(N);
        mp.act = G.act; mp.has_ln = G.has_ln; mp.eps = G.eps;
        const bool hb = G.bias >= 0, hr = G.res >= 0, hl = G.has_ln != 0;
        const int nc = static_cast<int>(N / 32);
        add(gi, 1, [=](const RunCtx& x) mutable {
          mp.X = reinterpret_cast<const float*>(x.resolve(pa));
          mp.W = reinterpret_cast<const float*>(x.resolve(pw));
          mp.bias = hb ? reinterpret_cast<const float*>(x.resolve(pb)) : nullptr;
          mp.R = hr ? reinterpret_cast<const float*>(x.resolve(pr)) : nullptr;
          mp.gamma = hl ? reinterpret_cast<const float*>(x.resolve(pg)) : nullptr;
          mp.beta = hl ? reinterpret_cast<const float*>(x.resolve(pbe)) : nullptr;
          mp.Y = reinterpret_cast<float*>(x.resolve(po));
          const int grid = std::min((mp.M + 7) / 8, 148 * 2);
          const size_t smem = (static_cast<size_t>(mp.K) * mp.N + 8 * mp.K) * sizeof(float);
          switch (nc) {
            case 1: { static bool once = (cudaFuncSetAttribute(k::fused_mlp_ln_f32<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024), true); (void)once; k::fused_mlp_ln_f32<1><<<grid, 256, smem, x.stream>>>(mp); break; }
            case 2: { static bool once = (cudaFuncSetAttribute(k::fused_mlp_ln_f32<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024), true); (void)once; k::fused_mlp_ln_f32<2><<<grid, 256, smem, x.stream>>>(mp); break; }
            case 3: { static bool once = (cudaFuncSetAttribute(k::fused_mlp_ln_f32<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024), true); (void)once; k::fused_mlp_ln_f32<3><<<grid, 256, smem, x.stream>>>(mp); break; }
            default: { static bool once = (cudaFuncSetAttribute(k::fused_mlp_ln_f32<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024), true); (void)once; k::fused_mlp_ln_f32<4><<<grid, 256, smem, x.stream>>>(mp); break; }
          }
          return cudaGetLastError();
        });
      }
      return OK;
    }
    // bf16 on tcgen05
    if (K % 64) return fail(E_UNSUPPORTED_OP, "bf16 GEMM needs K % 64 == 0 (k-chunk tensor maps)");
    if (lds[0] % 8 || lds[1] % 8 || N % 8 || (G.res >= 0 && lds[2] % 8)) return fail(E_UNSUPPORTED_OP, "GEMM operand rows must be 16-byte multiples");
    const bool lna = G.ln_a >= 0, lnr = G.ln_res >= 0, emit = G.emit_stats != 0;
    size_t pk = 0;
    bool pk_found = false;
    for (size_t i = 0; i < c.packed_consts.size(); ++i)
      if (c.packed_consts[i] == G.w) {
        const Compiled::PackedLn& e = c.packed_ln[i];
        if (lna ? (e.gamma == G.ln_gamma && e.beta == G.ln_beta && e.bias == G.bias) : e.gamma < 0) { pk = c.packed_off[i]; pk_found = true; }
      }
    if (!pk_found) return fail(E_INTERNAL, "no prepacked copy of " + W.name);
    if (G.has_ln) {
      // ---- GEMM (+bias, +residual) -> LayerNorm: K ranges of every 128x256 tile go to different CTAs,
      // which store their fp32 partial tiles into slabs of a workspace in the scratch region; the finishing
      // kernel adds a row's slabs in order, adds bias and residual and normalises.
      if (lds[1] != N || N > 1024) return fail(E_UNSUPPORTED_OP, "GEMM + LayerNorm: output rows must be contiguous and at most 1024 wide");
      Ptr pg = ptr_of(G.gamma, 0), pbe = ptr_of(G.beta, 0);
      const float eps = G.eps;
      const int ch = static_cast<int>((N / 8 + 31) / 32);
      for (auto& sg : segs) {
        if (sg.rows == 0) continue;
        Ptr pa = ptr_of(G.a, sg.r0), po = ptr_of(G.out, sg.r0), pr = G.res >= 0 ? ptr_of(G.res, sg.r0) : Ptr();
        Ptr pw; pw.where = 5; pw.off = static_cast<int64_t>(pk);
        Ptr pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
        const int M = static_cast<int>(sg.rows);
        const int64_t lda = lds[0], ldr = G.res >= 0 ? lds[2] : 0;
        const int tiles = ((M + 127) / 128) * static_cast<int>((N + 255) / 256);
        const int kstages = static_cast<int>(K / 64);
        // as many K ranges as fill the SMs once, at least four stages each
        int splits = std::max(1, std::min(148 / std::max(tiles, 1), kstages / 4));
        const int per = (kstages + splits - 1) / splits;
        splits = (kstages + per - 1) / per;
        const size_t ws_bytes = static_cast<size_t>(splits) * M * N * 4;
        scratch_need = std::max(scratch_need, ws_bytes);
        const bool hb = G.bias >= 0, hr = G.res >= 0;
        struct Cache { const void* a = nullptr; const void* w = nullptr; const void* o = nullptr; CUtensorMap ta, tb, to; };
        auto cache = std::make_shared<Cache>();
        add(gi, 2, [=](const RunCtx& x) {
          const void* A = x.resolve(pa);
          const void* Wt = x.resolve(pw);
          float* ws = reinterpret_cast<float*>(x.arena + x.plan->scratch_off[0]);
          if (cache->a != A || cache->w != Wt || cache->o != ws) {
            if (!encode_bf16_kchunks(&cache->ta, A, M, K, lda, 128, 1) || !encode_bf16_kchunks(&cache->tb, Wt, N, K, K, 256, 1) ||
                !encode_f32_slabs(&cache->to, ws, M, N, splits, 128))
              return cudaErrorInvalidValue;
            cache->a = A; cache->w = Wt; cache->o = ws;
          }
          k::GemmEpilogue ep{};
          ep.status = reinterpret_cast<int*>(x.arena);
          ep.splits = splits;
          ep.stages_per_split = per;
          const int grid = std::min(tiles * splits, x.plan->sm_count);
          constexpr int smem = k::GemmSmem<256, 1, 4>::TOTAL;
          static bool once = (cudaFuncSetAttribute(k::gemm_bf16_tcgen05<256, 1, 4, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);
          (void)once;
          launch_pdl(k::gemm_bf16_tcgen05<256, 1, 4, 0, true>, dim3(grid), dim3(k::GEMM_THREADS), smem, x.stream, cache->ta, cache->tb, cache->to,
                     cache->to, M, static_cast<int>(N), static_cast<int>(K), ep);
          auto* Bi = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
          auto* R = hr ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pr)) : nullptr;
          auto* Gm = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pg));
          auto* Bt = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pbe));
          auto* Y = reinterpret_cast<__nv_bfloat16*>(x.resolve(po));
          const long long rows = M;
          const unsigned lgrid = static_cast<unsigned>((rows + 7) / 8);
          switch (ch) {
            case 1: launch_pdl(k::splitk_ln_finish<1>, dim3(lgrid), dim3(256), 0, x.stream, static_cast<const float*>(ws), splits, Bi, R, static_cast<long long>(ldr), Gm, Bt, Y, rows, static_cast<int>(N), eps); break;
            case 2: launch_pdl(k::splitk_ln_finish<2>, dim3(lgrid), dim3(256), 0, x.stream, static_cast<const float*>(ws), splits, Bi, R, static_cast<long long>(ldr), Gm, Bt, Y, rows, static_cast<int>(N), eps); break;
            case 3: launch_pdl(k::splitk_ln_finish<3>, dim3(lgrid), dim3(256), 0, x.stream, static_cast<const float*>(ws), splits, Bi, R, static_cast<long long>(ldr), Gm, Bt, Y, rows, static_cast<int>(N), eps); break;
            default: launch_pdl(k::splitk_ln_finish<4>, dim3(lgrid), dim3(256), 0, x.stream, static_cast<const float*>(ws), splits, Bi, R, static_cast<long long>(ldr), Gm, Bt, Y, rows, static_cast<int>(N), eps); break;
          }
          return cudaGetLastError();
        });
      }
      return OK;
    }
    // folded LayerNorm: where the statistics of the normalised rows live, and where this group's own go
    if ((lna || lnr) && (lds[lna ? 0 : 2] != (lna ? K : N))) return fail(E_UNSUPPORTED_OP, "folded LayerNorm needs densely packed rows");
    if (emit && lds[1] != N) return fail(E_UNSUPPORTED_OP, "row statistics need densely packed output rows");
    if (p.stats_layout.size() != g.tensors.size()) p.stats_layout.assign(g.tensors.size(), Plan::StatsLayout());
    auto stats_ptr = [&](int t, int r0, int64_t width, Ptr* out, int64_t* pitch) -> bool {
      const int root = p.root_of[t];
      const RootBuf& RR = p.roots[root];
      if (RR.where != RootBuf::ARENA || RR.stats_off < 0 || p.views[t][r0].offset != 0) return false;
      const int64_t row0 = p.inst_off[root][r0] / (width * 2);
      out->where = RootBuf::ARENA;
      out->index = -1;
      out->off = static_cast<int64_t>(RR.arena_off) + RR.stats_off + row0 * 8;
      *pitch = RR.stats_rows;
      return true;
    };
    int bn_group = 0;   // a group that writes row statistics uses one tile width for all its launches
    for (auto& sg : segs) {
      if (sg.rows == 0) continue;
      Ptr pa = ptr_of(G.a, sg.r0), po = ptr_of(G.out, sg.r0), pr = G.res >= 0 ? ptr_of(G.res, sg.r0) : Ptr();
      Ptr pw; pw.where = 5; pw.off = static_cast<int64_t>(pk);
      Ptr pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
      const int M = static_cast<int>(sg.rows);
      const int64_t lda = lds[0], ldo = lds[1], ldr = G.res >= 0 ? lds[2] : 0;
      // Shape-class variant (the paper's multi-version idea, Section 4.4.2).  Two tile versions
      // exist: "fat" 128x256 tiles (one 64-wide k-chunk per stage) and "regular" 128x128 tiles (two
      // k-chunks per stage).  Pick the one with the smaller estimated makespan on the SMs: waves of
      // tiles times the per-tile main-loop time (stages x max(MMA, TMA) per stage).
      const int tiles_m = (M + 127) / 128;
      const int sms = 148;
      auto makespan = [&](int bn_, int kch) {
        const double tiles = static_cast<double>(tiles_m) * ((N + bn_ - 1) / bn_);
        const double waves = std::ceil(tiles / sms);
        const double stages = std::ceil(static_cast<double>(K) / (64.0 * kch));
        const double mma = kch * 4 * (bn_ / 2.0), floor_cycles = 540.0;
        const double tma = kch * (128 + bn_) * 128.0 / 70.0;   // empirical: stage cost grows with the operand bytes of a stage (measured 585 / 840 cycles)
        return waves * stages * std::max(std::max(mma, floor_cycles), tma);
      };
      int bn = (N > 128 && makespan(256, 1) <= makespan(128, 2)) ? 256 : 128;
      // Small problems: while 128x64 tiles still fit one wave, a CTA's time is pipeline fill + main loop +
      // epilogue of ONE tile, and both of the latter shrink with the tile (the epilogue is 0.6 us per 64 columns).
      if (bn == 128 && N > 64 && static_cast<int64_t>(tiles_m) * ((N + 63) / 64) <= sms) bn = 64;
      // the normalised-residual epilogue keeps three column vectors in shared memory (tiles up to 128 wide); row
      // statistics are written per whole tile width
      if (lnr && bn > 128) bn = 128;
      if (emit) {
        if (bn_group) bn = bn_group;
        while (bn > 64 && N % bn) bn /= 2;
        if (N % bn) return fail(E_UNSUPPORTED_OP, "row statistics need an output width that is a multiple of 64");
        bn_group = bn;
        p.stats_layout[G.out] = {static_cast<int>(N / bn) * 2, bn / 2};
      }
      // CTA pairs (tcgen05.mma.cta_group::2, 256 x BN tiles): each CTA loads its own A rows and half of the weight tile,
      // a third to a half fewer operand bytes per flop.  Same makespan estimate, per 64-wide k-chunk and pair of SMs.
      int pair_bn = 0;
      if ((c.flags & OPT_GEMM_PAIR) && !lna && !lnr && !emit && G.act2 == 0 && tiles_m >= 2 && N >= 128) {
        auto pair_span = [&](int bn_) {
          const double pairs = std::ceil(tiles_m / 2.0) * ((N + bn_ - 1) / bn_);
          const double waves = std::ceil(pairs / (sms / 2));
          const double mma = 4 * (bn_ / 2.0), tma = (128 + bn_ / 2) * 128.0 / 70.0;
          return waves * std::ceil(K / 64.0) * std::max(mma, tma);
        };
        const double single = bn == 256 ? makespan(256, 1) : makespan(128, 2);
        const int pb = (N >= 256 && pair_span(256) <= pair_span(128)) ? 256 : 128;
        static const bool force_pair = getenv("SOD2_GEMM_PAIR_FORCE") != nullptr;   // tests: the pair kernel wherever it is eligible
        if (pair_span(pb) < single || force_pair) pair_bn = pb;
      }
      const bool hb = G.bias >= 0, hr = G.res >= 0;
      const int act = G.act;
      const int act2 = G.act2;
      const int ln = lna ? 1 : lnr ? 2 : 0;
      Ptr ps_in, ps_out, pc1, pg, pbt;
      int64_t pitch_in = 0, pitch_out = 0;
      Plan::StatsLayout lay;
      if (ln) {
        const int raw = lna ? G.ln_a : G.ln_res;
        lay = p.stats_layout[raw];
        if (!lay.slots || !stats_ptr(raw, sg.r0, lna ? K : N, &ps_in, &pitch_in)) return fail(E_INTERNAL, "row statistics of " + g.tensors[raw].name + " are not planned");
        if (static_cast<int64_t>(lay.slots) * lay.cols != (lna ? K : N)) return fail(E_INTERNAL, "row statistics layout of " + g.tensors[raw].name);
        if (lna) { pc1.where = 5; pc1.off = static_cast<int64_t>(pk + ((static_cast<size_t>(N) * K * 2 + 255) & ~size_t(255))); }
        else { pg = ptr_of(G.ln_gamma, 0); pbt = ptr_of(G.ln_beta, 0); }
      }
      if (emit && !stats_ptr(G.out, sg.r0, N, &ps_out, &pitch_out)) return fail(E_INTERNAL, "row statistics of " + g.tensors[G.out].name + " are not planned");
      const float ln_eps = G.ln_eps;
      struct Cache { const void* a = nullptr; const void* w = nullptr; const void* o = nullptr; const void* r = nullptr; CUtensorMap ta, tb, to, tr; };
      auto cache = std::make_shared<Cache>();
      add(gi, 1, [=](const RunCtx& x) {
        const void* A = x.resolve(pa);
        const void* Wt = x.resolve(pw);
        void* O = x.resolve(po);
        const void* R = hr ? x.resolve(pr) : O;
        if (cache->a != A || cache->w != Wt || cache->o != O || cache->r != R) {
          const int kch = pair_bn ? (pair_bn == 256 ? 1 : 2) : (bn == 256 ? 1 : 2);
          const int brows = pair_bn ? pair_bn / 2 : bn;      // a CTA of a pair loads half of the weight tile
          if (!encode_bf16_kchunks(&cache->ta, A, M, K, lda, 128, kch) || !encode_bf16_kchunks(&cache->tb, Wt, N, K, K, brows, kch) ||
              !encode_bf16_2d(&cache->to, O, M, N, ldo, 128) || !encode_bf16_2d(&cache->tr, R, M, N, hr ? ldr : ldo, 128))
            return cudaErrorInvalidValue;
          cache->a = A; cache->w = Wt; cache->o = O; cache->r = R;
        }
        k::GemmEpilogue ep{};
        ep.bias = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
        ep.has_residual = hr;
        ep.act2 = act2;
        ep.status = reinterpret_cast<int*>(x.arena);
        if (ln) {
          ep.ln_stats = reinterpret_cast<const float2*>(x.resolve(ps_in));
          ep.ln_pitch = pitch_in;
          ep.ln_slots = lay.slots;
          ep.ln_cols = lay.cols;
          ep.ln_eps = ln_eps;
          if (ln == 1) {
            ep.ln_c1 = reinterpret_cast<const float*>(x.resolve(pc1));
            ep.ln_c2 = ep.ln_c1 + N;
          } else {
            ep.ln_gamma = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pg));
            ep.ln_beta = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pbt));
          }
        }
        if (emit) {
          ep.emit_stats = reinterpret_cast<float2*>(x.resolve(ps_out));
          ep.emit_pitch = pitch_out;
        }
        const int Ni = static_cast<int>(N), Ki = static_cast<int>(K);
        if (pair_bn) {
          const int pairs = ((tiles_m + 1) / 2) * static_cast<int>((N + pair_bn - 1) / pair_bn);
          const dim3 gp(2 * std::max(1, std::min(pairs, x.plan->sm_count / 2)));
          const cudaError_t ep2 = pair_bn == 256 ? gemm_pair_dispatch<256, 1, 6>(act, hr, gp, x.stream, cache->ta, cache->tb, cache->to, cache->tr, M, Ni, Ki, ep)
                                                 : gemm_pair_dispatch<128, 2, 4>(act, hr, gp, x.stream, cache->ta, cache->tb, cache->to, cache->tr, M, Ni, Ki, ep);
          return ep2 != cudaSuccess ? ep2 : cudaGetLastError();
        }
        const int tiles = tiles_m * static_cast<int>((N + bn - 1) / bn);
        const int grid = std::min(tiles, x.plan->sm_count);
        const dim3 gd(grid);
        cudaError_t e;
        if (bn == 256) e = gemm_dispatch<256, 1, 4>(act, hr, ln, emit, gd, x.stream, cache->ta, cache->tb, cache->to, cache->tr, M, Ni, Ki, ep);
        else if (bn == 128) e = gemm_dispatch<128, 2, 3>(act, hr, ln, emit, gd, x.stream, cache->ta, cache->tb, cache->to, cache->tr, M, Ni, Ki, ep);
        else e = gemm_dispatch<64, 2, 3>(act, hr, ln, emit, gd, x.stream, cache->ta, cache->tb, cache->to, cache->tr, M, Ni, Ki, ep);
        return e != cudaSuccess ? e : cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ GEMM chains
  // Epilogue version of the chain kernel for a group, or -1 if the group cannot be a chain member.
  int chain_epi(const Group& G) const {
    if (G.kind != GKind::GEMM || G.has_ln || G.act2 || g.tensors[G.a].dtype != DType::BF16) return -1;
    const bool res = G.res >= 0, emit = G.emit_stats != 0;
    const int ln = G.ln_a >= 0 ? 1 : G.ln_res >= 0 ? 2 : 0;
    if (G.act == 0 && !res && ln == 0 && !emit) return k::CE_PLAIN;
    if (G.act == 0 && res && ln == 0 && !emit) return k::CE_RES;
    if (G.act == 1 && !res && ln == 0 && !emit) return k::CE_GELU;
    if (G.act == 0 && res && ln == 0 && emit) return k::CE_RES_EMIT;
    if (G.act == 0 && res && ln == 2 && !emit) return k::CE_RES_LN2;
    if (G.act == 0 && res && ln == 2 && emit) return k::CE_RES_LN2_EMIT;
    if (G.act == 0 && !res && ln == 1 && !emit) return k::CE_LN1;
    if (G.act == 1 && !res && ln == 1 && !emit) return k::CE_LN1_GELU;
    return -1;
  }
  struct ChainMember { int64_t M = 0, N = 0, K = 0, lda = 0, ldo = 0, ldr = 0; int epi = -1; };
  // A group as a chain member: one launch segment over all requests, shapes the 128 x 128 tile version takes.
  bool chain_member(const Group& G, ChainMember* cm) {
    cm->epi = chain_epi(G);
    if (cm->epi < 0) return false;
    const Tensor& W = g.tensors[G.w];
    cm->K = W.S.dims[0].e.const_value();
    cm->N = W.S.dims[1].e.const_value();
    std::vector<int> ts = {G.a, G.out};
    if (G.res >= 0) ts.push_back(G.res);
    int64_t cols;
    std::vector<int64_t> lds;
    std::vector<Seg> segs;
    const std::string keep = p.err;
    if (row_segments(ts, &cols, &lds, &segs) != OK) { p.err = keep; return false; }
    if (segs.size() != 1 || segs[0].rows <= 0 || cols != cm->K) return false;
    if (cm->K % 64 || lds[0] % 8 || lds[1] % 8 || cm->N % 8 || (G.res >= 0 && lds[2] % 8)) return false;
    if (G.emit_stats && (cm->N % 128 || lds[1] != cm->N)) return false;
    if (G.ln_a >= 0 && lds[0] != cm->K) return false;
    if (G.ln_res >= 0 && lds[2] != cm->N) return false;
    cm->M = segs[0].rows;
    cm->lda = lds[0]; cm->ldo = lds[1]; cm->ldr = G.res >= 0 ? lds[2] : 0;
    return true;
  }
  // the same bytes in the same order: root, offset, extents and strides of request 0 (the members are one segment)
  bool same_view(int t1, int t2) const {
    const View &a = p.views[t1][0], &b = p.views[t2][0];
    return p.root_of[t1] == p.root_of[t2] && a.offset == b.offset && a.dims == b.dims && a.strides == b.strides;
  }
  // Maximal runs of consecutive chainable GEMM groups with equal row counts.  A member may read rows written by an
  // earlier member only as its A operand or its residual and only as the very view the earlier member wrote
  // (row block i then depends on row block i alone); any other overlap ends the run.
  Status find_chains() {
    p.chains.clear();
    p.chain_of.assign(c.groups.size(), -1);
    p.chain_counter_words = 0;
    if (!(c.flags & OPT_GEMM_CHAIN) || (c.flags & OPT_NO_FUSION)) return OK;
    size_t gi = 0;
    while (gi < c.groups.size()) {
      ChainMember first;
      if (!chain_member(c.groups[gi], &first)) { ++gi; continue; }
      std::vector<int> run = {static_cast<int>(gi)};
      size_t gj = gi + 1;
      static const int chain_max = [] { const char* e = getenv("SOD2_CHAIN_MAX"); const int v = e ? atoi(e) : k::CHAIN_MAX; return std::max(1, std::min(v, k::CHAIN_MAX)); }();
      while (gj < c.groups.size() && run.size() < static_cast<size_t>(chain_max)) {
        ChainMember cm;
        const Group& G = c.groups[gj];
        if (!chain_member(G, &cm) || cm.M != first.M) break;
        bool ok = true;
        for (int t : G.ext_in) {
          if (g.tensors[t].kind == TKind::CONST || c.storage[t].kind == Storage::FOLDED || p.views[t].empty()) continue;
          for (int m : run) {
            const int o = c.groups[m].out;
            if (p.root_of[t] != p.root_of[o]) continue;
            if (!((t == G.a || t == G.res) && same_view(t, o))) ok = false;
          }
        }
        // nothing a member writes may be storage an earlier member reads or writes
        for (int m : run) {
          const Group& E = c.groups[m];
          for (int t : E.ext_in) if (!p.views[t].empty() && p.root_of[t] == p.root_of[G.out]) ok = false;
          if (p.root_of[E.out] == p.root_of[G.out]) ok = false;
        }
        if (!ok) break;
        run.push_back(static_cast<int>(gj));
        ++gj;
      }
      if (run.size() >= 2) {
        Plan::Chain ch;
        ch.groups = run;
        ch.rows = static_cast<int>(first.M);
        ch.counter_word = p.chain_counter_words;
        p.chain_counter_words += run.size() * static_cast<size_t>((first.M + 127) / 128);
        for (int m : run) p.chain_of[m] = static_cast<int>(p.chains.size());
        p.chains.push_back(ch);
        gi = gj;
      } else {
        ++gi;
      }
    }
    return OK;
  }

  // One launch for all members of chain `ci`.
  Status build_gemm_chain(int ci) {
    const Plan::Chain& ch = p.chains[ci];
    const int n = static_cast<int>(ch.groups.size());
    if (p.stats_layout.size() != g.tensors.size()) p.stats_layout.assign(g.tensors.size(), Plan::StatsLayout());
    struct Mem {
      ChainMember cm;
      Ptr pa, po, pr, pw, pb, pc1, pg, pbt, ps_in, ps_out;
      int64_t pitch_in = 0, pitch_out = 0;
      Plan::StatsLayout lay;
      bool hb = false, hr = false, emit = false;
      int ln = 0, dep_a = -1, dep_r = -1;
      float eps = 1e-5f;
    };
    std::vector<Mem> ms(n);
    auto stats_ptr = [&](int t, int64_t width, Ptr* out, int64_t* pitch) -> bool {
      const int root = p.root_of[t];
      const RootBuf& RR = p.roots[root];
      if (RR.where != RootBuf::ARENA || RR.stats_off < 0 || p.views[t][0].offset != 0) return false;
      const int64_t row0 = p.inst_off[root][0] / (width * 2);
      out->where = RootBuf::ARENA;
      out->index = -1;
      out->off = static_cast<int64_t>(RR.arena_off) + RR.stats_off + row0 * 8;
      *pitch = RR.stats_rows;
      return true;
    };
    double flops_total = 0.0;
    std::vector<double> fl(n);
    for (int i = 0; i < n; ++i) {
      const Group& G = c.groups[ch.groups[i]];
      Mem& m = ms[i];
      if (!chain_member(G, &m.cm)) return fail(E_INTERNAL, "chain member changed its mind");
      const int64_t N = m.cm.N, K = m.cm.K;
      m.hb = G.bias >= 0; m.hr = G.res >= 0; m.emit = G.emit_stats != 0;
      m.ln = G.ln_a >= 0 ? 1 : G.ln_res >= 0 ? 2 : 0;
      m.eps = G.ln_eps;
      m.pa = ptr_of(G.a, 0); m.po = ptr_of(G.out, 0);
      if (m.hr) m.pr = ptr_of(G.res, 0);
      if (m.hb) m.pb = ptr_of(G.bias, 0);
      size_t pk = 0;
      bool found = false;
      for (size_t q = 0; q < c.packed_consts.size(); ++q)
        if (c.packed_consts[q] == G.w) {
          const Compiled::PackedLn& e = c.packed_ln[q];
          if (m.ln == 1 ? (e.gamma == G.ln_gamma && e.beta == G.ln_beta && e.bias == G.bias) : e.gamma < 0) { pk = c.packed_off[q]; found = true; }
        }
      if (!found) return fail(E_INTERNAL, "no prepacked copy of " + g.tensors[G.w].name);
      m.pw.where = 5; m.pw.off = static_cast<int64_t>(pk);
      if (m.emit) {
        p.stats_layout[G.out] = {static_cast<int>(N / k::CHAIN_BN) * 2, k::CHAIN_BN / 2};
        if (!stats_ptr(G.out, N, &m.ps_out, &m.pitch_out)) return fail(E_INTERNAL, "row statistics of " + g.tensors[G.out].name + " are not planned");
      }
      if (m.ln) {
        const int raw = m.ln == 1 ? G.ln_a : G.ln_res;
        m.lay = p.stats_layout[raw];
        if (!m.lay.slots || !stats_ptr(raw, m.ln == 1 ? K : N, &m.ps_in, &m.pitch_in)) return fail(E_INTERNAL, "row statistics of " + g.tensors[raw].name + " are not planned");
        if (static_cast<int64_t>(m.lay.slots) * m.lay.cols != (m.ln == 1 ? K : N)) return fail(E_INTERNAL, "row statistics layout of " + g.tensors[raw].name);
        if (m.ln == 1) { m.pc1.where = 5; m.pc1.off = static_cast<int64_t>(pk + ((static_cast<size_t>(N) * K * 2 + 255) & ~size_t(255))); }
        else { m.pg = ptr_of(G.ln_gamma, 0); m.pbt = ptr_of(G.ln_beta, 0); }
      }
      for (int j = 0; j < i; ++j) {
        const int o = c.groups[ch.groups[j]].out;
        if (p.root_of[G.a] == p.root_of[o]) m.dep_a = j;
        if (m.hr && p.root_of[G.res] == p.root_of[o]) m.dep_r = j;
      }
      fl[i] = 2.0 * static_cast<double>(m.cm.M) * N * K;
      flops_total += fl[i];
    }
    const int M = ch.rows;
    const int tiles_m = (M + 127) / 128;
    const size_t counter_off = p.chain_counter_off + 4 * ch.counter_word;   // chain_counter_off is final: the arena is planned
    struct Cache { std::vector<const void*> key; k::GemmChainMaps maps; };
    auto cache = std::make_shared<Cache>();
    auto L = std::make_shared<Launch>();
    L->group = ch.groups[0];
    L->n_kernels = 1;
    for (int i = 0; i < n; ++i) L->share.push_back({ch.groups[i], flops_total > 0 ? fl[i] / flops_total : 1.0 / n});
    L->fn = [=](const RunCtx& x) {
      std::vector<const void*> key;
      k::GemmChainParams cp{};
      cp.n = n; cp.M = M; cp.tiles_m = tiles_m;
      cp.done = reinterpret_cast<unsigned*>(x.arena + counter_off);
      int tile0 = 0;
      const void* A[k::CHAIN_MAX]; const void* Wt[k::CHAIN_MAX]; void* O[k::CHAIN_MAX]; const void* R[k::CHAIN_MAX];
      for (int i = 0; i < n; ++i) {
        const Mem& m = ms[i];
        A[i] = x.resolve(m.pa); Wt[i] = x.resolve(m.pw); O[i] = x.resolve(m.po); R[i] = m.hr ? x.resolve(m.pr) : O[i];
        key.push_back(A[i]); key.push_back(Wt[i]); key.push_back(O[i]); key.push_back(R[i]);
        k::GemmChainProblem& P = cp.p[i];
        P.N = static_cast<int>(m.cm.N); P.K = static_cast<int>(m.cm.K);
        P.tiles_n = static_cast<int>((m.cm.N + k::CHAIN_BN - 1) / k::CHAIN_BN);
        P.tile0 = tile0;
        tile0 += tiles_m * P.tiles_n;
        P.epi = m.cm.epi; P.dep_a = m.dep_a; P.dep_r = m.dep_r;
        P.ep.bias = m.hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(m.pb)) : nullptr;
        P.ep.has_residual = m.hr;
        P.ep.status = reinterpret_cast<int*>(x.arena);
        if (m.ln) {
          P.ep.ln_stats = reinterpret_cast<const float2*>(x.resolve(m.ps_in));
          P.ep.ln_pitch = m.pitch_in; P.ep.ln_slots = m.lay.slots; P.ep.ln_cols = m.lay.cols; P.ep.ln_eps = m.eps;
          if (m.ln == 1) { P.ep.ln_c1 = reinterpret_cast<const float*>(x.resolve(m.pc1)); P.ep.ln_c2 = P.ep.ln_c1 + m.cm.N; }
          else { P.ep.ln_gamma = reinterpret_cast<const __nv_bfloat16*>(x.resolve(m.pg)); P.ep.ln_beta = reinterpret_cast<const __nv_bfloat16*>(x.resolve(m.pbt)); }
        }
        if (m.emit) { P.ep.emit_stats = reinterpret_cast<float2*>(x.resolve(m.ps_out)); P.ep.emit_pitch = m.pitch_out; }
      }
      cp.total_tiles = tile0;
      if (cache->key != key) {
        for (int i = 0; i < n; ++i) {
          const Mem& m = ms[i];
          if (!encode_bf16_kchunks(&cache->maps.a[i], A[i], M, m.cm.K, m.cm.lda, 128, k::CHAIN_KCH) ||
              !encode_bf16_kchunks(&cache->maps.b[i], Wt[i], m.cm.N, m.cm.K, m.cm.K, k::CHAIN_BN, k::CHAIN_KCH) ||
              !encode_bf16_2d(&cache->maps.o[i], O[i], M, m.cm.N, m.cm.ldo, 128) ||
              !encode_bf16_2d(&cache->maps.r[i], R[i], M, m.cm.N, m.hr ? m.cm.ldr : m.cm.ldo, 128))
            return cudaErrorInvalidValue;
        }
        for (int i = n; i < k::CHAIN_MAX; ++i) { cache->maps.a[i] = cache->maps.a[0]; cache->maps.b[i] = cache->maps.b[0]; cache->maps.o[i] = cache->maps.o[0]; cache->maps.r[i] = cache->maps.r[0]; }
        cache->key = key;
      }
      constexpr int smem = k::GemmSmem<k::CHAIN_BN, k::CHAIN_KCH, k::CHAIN_STAGES>::TOTAL;
      static bool once = (cudaFuncSetAttribute(k::gemm_chain_bf16_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);
      (void)once;
      const int grid = std::min(cp.total_tiles, x.plan->sm_count);
      const cudaError_t e = launch_pdl(k::gemm_chain_bf16_tcgen05, dim3(grid), dim3(k::GEMM_THREADS), smem, x.stream, cache->maps, cp,
                                       reinterpret_cast<int*>(x.arena));
      return e != cudaSuccess ? e : cudaGetLastError();
    };
    p.gpu_launches += 1;
    p.launches.push_back(L);
    return OK;
  }

  // ------------------------------------------------------------------------------ attention
  Status build_attention(int gi, const Group& G) {
    if (g.tensors[G.q].dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "attention group is bf16 only");
    for (int r0 = 0; r0 < p.n_req; r0 += k::ATTN_MAX_REQ) {
      const int nr = std::min(k::ATTN_MAX_REQ, p.n_req - r0);
      k::AttnParams ap{};
      ap.n_req = nr;
      ap.scale_log2e = G.scale * 1.4426950408889634f;
      Ptr bq = ptr_of(G.q, r0), bk = ptr_of(G.k, r0), bv = ptr_of(G.v, r0), bo = ptr_of(G.out, r0);
      int tiles = 0, H = -1;
      for (int i = 0; i < nr; ++i) {
        const int r = r0 + i;
        const View &q = p.views[G.q][r], &kk = p.views[G.k][r], &v = p.views[G.v][r], &o = p.views[G.out][r];
        const int rk = static_cast<int>(q.dims.size());
        if (rk < 3 || kk.dims.size() != q.dims.size() || v.dims.size() != q.dims.size()) return fail(E_UNSUPPORTED_OP, "attention operands need rank >= 3");
        for (int d = 0; d < rk - 3; ++d) if (q.dims[d] != 1) return fail(E_UNSUPPORTED_OP, "attention: leading batch dims must be 1");
        const int64_t h = q.dims[rk - 3], L = q.dims[rk - 2], dh = q.dims[rk - 1];
        if (dh != 64) return fail(E_UNSUPPORTED_OP, "attention kernel is specialised for head dim 64");
        if (kk.dims[rk - 2] != dh || kk.dims[rk - 1] != L || v.dims[rk - 2] != L || v.dims[rk - 1] != dh) return fail(E_SHAPE_CONFLICT, "attention operand shapes");
        if (q.strides[rk - 1] != 1 || kk.strides[rk - 2] != 1 || v.strides[rk - 1] != 1 || o.strides[rk - 1] != 1) return fail(E_UNSUPPORTED_OP, "attention: head dim must be contiguous");
        if (H < 0) H = static_cast<int>(h); else if (H != h) return fail(E_UNSUPPORTED_OP, "attention: head count differs");
        k::AttnReq& R = ap.r[i];
        Ptr pq = ptr_of(G.q, r), pk2 = ptr_of(G.k, r), pv = ptr_of(G.v, r), po = ptr_of(G.out, r);
        if (!same_base(pq, bq) || !same_base(pk2, bk) || !same_base(pv, bv) || !same_base(po, bo)) return fail(E_INTERNAL, "attention bases");
        R.q_off = (pq.off - bq.off) / 2; R.k_off = (pk2.off - bk.off) / 2; R.v_off = (pv.off - bv.off) / 2; R.o_off = (po.off - bo.off) / 2;
        R.L = static_cast<int>(L);
        R.q_ts = static_cast<int>(q.strides[rk - 2]); R.k_ts = static_cast<int>(kk.strides[rk - 1]);
        R.v_ts = static_cast<int>(v.strides[rk - 2]); R.o_ts = static_cast<int>(o.strides[rk - 2]);
        R.q_hs = static_cast<int>(q.strides[rk - 3]); R.k_hs = static_cast<int>(kk.strides[rk - 3]);
        R.v_hs = static_cast<int>(v.strides[rk - 3]); R.o_hs = static_cast<int>(o.strides[rk - 3]);
        if ((R.q_ts | R.k_ts | R.v_ts | R.q_hs | R.k_hs | R.v_hs) % 8 || (pq.off | pk2.off | pv.off) % 16 || (R.o_ts | R.o_hs) % 2 || po.off % 4)
          return fail(E_MISALIGNED, "attention operands must be 16-byte aligned");
        ap.tile_start[i] = tiles;
        tiles += static_cast<int>((L + 63) / 64);
      }
      ap.tile_start[nr] = tiles;
      ap.H = H;
      if (tiles == 0) continue;
      // tcgen05 path: needs Q, K, V as 2-D [token, column] maps over one packed buffer each (the same
      // token stride, head stride and head-0 column for every request, rows in increasing order)
      {
        k::AtcParams tp{};
        bool ok = !(c.flags & OPT_LEGACY_ATTENTION);
        auto split = [&](long long off, int ts, int* row, int* col) { if (off < 0 || ts <= 0) { ok = false; return; } *row = static_cast<int>(off / ts); *col = static_cast<int>(off % ts); };
        const k::AttnReq& R0 = ap.r[0];
        int order[k::ATTN_MAX_REQ];
        for (int i = 0; i < nr; ++i) order[i] = i;
        std::stable_sort(order, order + nr, [&](int a, int b) { return ap.r[a].L > ap.r[b].L; });
        long long rows_q = 0, rows_k = 0, rows_v = 0;
        int tiles128 = 0;
        for (int s = 0; s < nr && ok; ++s) {
          const k::AttnReq& R = ap.r[order[s]];
          if (R.q_ts != R0.q_ts || R.k_ts != R0.k_ts || R.v_ts != R0.v_ts || R.q_hs != R0.q_hs || R.k_hs != R0.k_hs || R.v_hs != R0.v_hs ||
              R.o_ts != R0.o_ts || R.o_hs != R0.o_hs || (R.o_ts | R.o_hs) % 8 || R.o_off % 8) { ok = false; break; }
          k::AtcReq& T = tp.r[s];
          int cq = 0, ck = 0, cv = 0;
          split(R.q_off, R.q_ts, &T.q_row, &cq); split(R.k_off, R.k_ts, &T.k_row, &ck); split(R.v_off, R.v_ts, &T.v_row, &cv);
          if (!ok) break;
          if (s == 0) { tp.q_col = cq; tp.k_col = ck; tp.v_col = cv; }
          if (cq != tp.q_col || ck != tp.k_col || cv != tp.v_col) { ok = false; break; }
          T.L = R.L; T.o_off = R.o_off;
          rows_q = std::max<long long>(rows_q, T.q_row + R.L); rows_k = std::max<long long>(rows_k, T.k_row + R.L); rows_v = std::max<long long>(rows_v, T.v_row + R.L);
          tp.tile_start[s] = tiles128;
          tiles128 += (R.L + 127) / 128;
        }
        tp.tile_start[nr] = tiles128;
        if (ok && (tp.q_col + (H - 1) * R0.q_hs + 64 > R0.q_ts || tp.k_col + (H - 1) * R0.k_hs + 64 > R0.k_ts || tp.v_col + (H - 1) * R0.v_hs + 64 > R0.v_ts ||
                   (tp.q_col | tp.k_col | tp.v_col) % 8 || bo.off % 16 || !(G.scale > 0.f)))
          ok = false;
        if (ok) {
          tp.n_req = nr; tp.H = H;
          tp.q_hs = R0.q_hs; tp.k_hs = R0.k_hs; tp.v_hs = R0.v_hs; tp.o_ts = R0.o_ts; tp.o_hs = R0.o_hs;
          tp.scale_log2e = ap.scale_log2e;
          const int q_ts = R0.q_ts, k_ts = R0.k_ts, v_ts = R0.v_ts;
          struct Cache { const void* q = nullptr; const void* k = nullptr; const void* v = nullptr; CUtensorMap tq, tk, tv; };
          auto cache = std::make_shared<Cache>();
          add(gi, 1, [=](const RunCtx& x) mutable {
            const void* Q = x.resolve(bq);
            const void* Kp = x.resolve(bk);
            const void* V = x.resolve(bv);
            if (cache->q != Q || cache->k != Kp || cache->v != V) {
              if (!encode_bf16_2d(&cache->tq, Q, rows_q, q_ts, q_ts, 128) || !encode_bf16_2d(&cache->tk, Kp, rows_k, k_ts, k_ts, k::ATC_KB) ||
                  !encode_bf16_2d(&cache->tv, V, rows_v, v_ts, v_ts, k::ATC_KB))
                return cudaErrorInvalidValue;
              cache->q = Q; cache->k = Kp; cache->v = V;
            }
            tp.o = reinterpret_cast<__nv_bfloat16*>(x.resolve(bo));
            tp.status = reinterpret_cast<int*>(x.arena);
            static bool once = (cudaFuncSetAttribute(k::attention_tcgen05_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, k::ATC_SMEM), true);
            (void)once;
            launch_pdl(k::attention_tcgen05_bf16, dim3(static_cast<unsigned>(tiles128) * tp.H), dim3(k::ATC_THREADS), k::ATC_SMEM, x.stream,
                       cache->tq, cache->tk, cache->tv, tp);
            return cudaGetLastError();
          });
          continue;
        }
      }
      add(gi, 1, [=](const RunCtx& x) mutable {
        ap.q = reinterpret_cast<const __nv_bfloat16*>(x.resolve(bq));
        ap.k = reinterpret_cast<const __nv_bfloat16*>(x.resolve(bk));
        ap.v = reinterpret_cast<const __nv_bfloat16*>(x.resolve(bv));
        ap.o = reinterpret_cast<__nv_bfloat16*>(x.resolve(bo));
        launch_pdl(k::attention_fwd_bf16, dim3(tiles, ap.H), dim3(128), 0, x.stream, ap);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ LayerNorm rows
  Status build_layernorm(int gi, const Group& G) {
    int64_t D;
    std::vector<int64_t> lds;
    std::vector<Seg> segs;
    Status s = row_segments({G.a, G.out}, &D, &lds, &segs);
    if (s != OK) return s;
    if (lds[0] != D || lds[1] != D || D % 8 || D > 1024) return build_chain(gi, G, true);
    // the row kernel reads gamma and beta before it waits for the previous kernel: they must be constants
    if (g.tensors[G.gamma].kind != TKind::CONST || g.tensors[G.beta].kind != TKind::CONST) return build_chain(gi, G, true);
    Ptr pg = ptr_of(G.gamma, 0), pb = ptr_of(G.beta, 0);
    const float eps = G.eps;
    const int ch = static_cast<int>((D / 8 + 31) / 32);
    for (auto& sg : segs) {
      if (!sg.rows) continue;
      Ptr pa = ptr_of(G.a, sg.r0), po = ptr_of(G.out, sg.r0);
      const long long rows = sg.rows;
      add(gi, 1, [=](const RunCtx& x) {
        auto* X = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pa));
        auto* Y = reinterpret_cast<__nv_bfloat16*>(x.resolve(po));
        auto* Gm = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pg));
        auto* Bt = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb));
        const unsigned grid = static_cast<unsigned>((rows + 7) / 8);
        const bool full = D == ch * 256;
#define SOD2_LN_CASE(CH_)                                                                                                 \
        case CH_:                                                                                                        \
          if (full) launch_pdl(k::layernorm_bf16<CH_, true>, dim3(grid), dim3(256), 0, x.stream, X, Gm, Bt, Y, rows, static_cast<int>(D), eps); \
          else launch_pdl(k::layernorm_bf16<CH_, false>, dim3(grid), dim3(256), 0, x.stream, X, Gm, Bt, Y, rows, static_cast<int>(D), eps);     \
          break;
        switch (ch) {
          SOD2_LN_CASE(1)
          SOD2_LN_CASE(2)
          SOD2_LN_CASE(3)
          default:
          SOD2_LN_CASE(4)
        }
#undef SOD2_LN_CASE
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ generic chain
  // The requests of a batch go through one launch (a request table of up to CHAIN_MAX_REQ entries; a new launch
  // starts when the table is full or a request's operand lies in another buffer than the table's).
  Status build_chain(int gi, const Group& G, bool ln_only = false) {
    const Tensor& O = g.tensors[G.out];
    if (O.S.rank > 4) return fail(E_UNSUPPORTED_OP, "chain kernel supports rank <= 4");
    const int n_ops = ln_only ? 0 : static_cast<int>(G.chain_ops.size());
    const int red = ln_only ? 2 : G.red;
    // operand k: 0 = in0, 1 + i = operand of operator i (absent for unary operators)
    std::vector<int> opnd(1 + k::CHAIN_MAX_OPS, -1);
    opnd[0] = G.a;
    for (int i = 0; i < n_ops; ++i) opnd[1 + i] = G.chain_operands[i];
    k::ChainBatch proto{};
    proto.n_ops = n_ops;
    for (int i = 0; i < n_ops; ++i) proto.op[i] = G.chain_ops[i];
    proto.out_bf16 = O.dtype == DType::BF16;
    proto.red = red;
    proto.eps = G.eps;
    proto.gb_bf16 = red == 2 ? g.tensors[G.gamma].dtype == DType::BF16 : 0;
    for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx)
      if (opnd[kx] >= 0) {
        const Tensor& T = g.tensors[opnd[kx]];
        proto.is_bf16[kx] = T.dtype == DType::BF16;
        if (T.kind == TKind::FCONST) proto.scalar[kx] = static_cast<float>(T.fdata);
      }
    Ptr pg = red == 2 ? ptr_of(G.gamma, 0) : Ptr(), pb = red == 2 ? ptr_of(G.beta, 0) : Ptr();
    // operands read through a pointer (the launch closures outlive this builder: they capture plain values only)
    std::vector<char> has_ptr(1 + k::CHAIN_MAX_OPS, 0);
    for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx) has_ptr[kx] = opnd[kx] >= 0 && g.tensors[opnd[kx]].kind != TKind::FCONST;
    struct Pending {
      k::ChainBatch cb;
      std::vector<Ptr> base;      // per operand: pointer of the table's first request
      Ptr out;
      bool vec = true;            // every request qualifies for the 8-wide kernel
      bool vec16 = true;          // ... and has a last extent that is a multiple of 16
      int max_cols = 0;
    };
    auto fresh = [&]() { Pending q; q.cb = proto; q.base.assign(1 + k::CHAIN_MAX_OPS, Ptr()); return q; };
    Pending cur = fresh();
    auto flush = [&]() {
      if (!cur.cb.n_req) return;
      Pending q = cur;
      cur = fresh();
      add(gi, 1, [=](const RunCtx& x) mutable {
        k::ChainBatch& cb = q.cb;
        for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx)
          cb.base[kx] = has_ptr[kx] ? x.resolve(q.base[kx]) : nullptr;
        cb.out = x.resolve(q.out);
        if (red == 2) { cb.gamma = x.resolve(pg); cb.beta = x.resolve(pb); }
        if (!red) {
          const unsigned grid = static_cast<unsigned>(std::max<long long>(1, std::min<long long>((cb.total + 255) / 256, 148 * 32)));
          if (q.vec && q.vec16) {
            // two vectors per item: the table was filled in units of 8 elements
            for (int i = 0; i < cb.n_req; ++i) cb.r[i].first /= 2;
            cb.total /= 2;
            const unsigned g16 = static_cast<unsigned>(std::max<long long>(1, std::min<long long>((cb.total + 255) / 256, 148 * 32)));
            k::chain_elementwise_vec<2><<<g16, 256, 0, x.stream>>>(cb);
            for (int i = 0; i < cb.n_req; ++i) cb.r[i].first *= 2;
            cb.total *= 2;
          } else if (q.vec) k::chain_elementwise_vec<1><<<grid, 256, 0, x.stream>>>(cb);
          else k::chain_elementwise<<<grid, 256, 0, x.stream>>>(cb);
        } else if (q.max_cols <= k::ROWRED_WARP_COLS) {
          const size_t smem = static_cast<size_t>(q.max_cols) * 4 * 8;
          if (smem > 48 * 1024) { static bool once = (cudaFuncSetAttribute(k::chain_rowreduce_warp, cudaFuncAttributeMaxDynamicSharedMemorySize, k::ROWRED_WARP_COLS * 32), true); (void)once; }
          const unsigned grid = static_cast<unsigned>(std::max<long long>(1, std::min<long long>((cb.total + 7) / 8, 148 * 8)));
          k::chain_rowreduce_warp<<<grid, 256, smem, x.stream>>>(cb, q.max_cols);
        } else {
          const size_t smem = static_cast<size_t>(q.max_cols) * 4;
          if (smem > 48 * 1024) { static bool once = (cudaFuncSetAttribute(k::chain_rowreduce, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024), true); (void)once; }
          k::chain_rowreduce<<<static_cast<unsigned>(std::max<long long>(1, std::min<long long>(cb.total, 148 * 8))), 256, smem, x.stream>>>(cb);
        }
        return cudaGetLastError();
      });
    };
    for (int r = 0; r < p.n_req; ++r) {
      const View& ov = p.views[G.out][r];
      if (!ov.contiguous()) return fail(E_UNSUPPORTED_OP, "chain output must be contiguous");
      if (numel(ov.dims) == 0) continue;
      int64_t od[4] = {1, 1, 1, 1};
      for (size_t i = 0; i < ov.dims.size(); ++i) od[4 - ov.dims.size() + i] = ov.dims[i];
      for (int i = 0; i < 4; ++i) if (od[i] >= (int64_t(1) << 31)) return fail(E_UNSUPPORTED_OP, "chain extent above 2^31");
      if (red && od[3] * 4 > 200 * 1024) return fail(E_UNSUPPORTED_OP, "row too long for the row-reduction kernel");
      // this request's operands: pointer, strides (0 on broadcast dims: read in place)
      std::vector<Ptr> ptrs(1 + k::CHAIN_MAX_OPS);
      int strides[1 + k::CHAIN_MAX_OPS][4] = {};
      for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx) {
        const int t = opnd[kx];
        if (t < 0 || g.tensors[t].kind == TKind::FCONST) continue;
        const int rr = g.tensors[t].kind == TKind::CONST ? 0 : r;
        const View& v = p.views[t][rr];
        const int rk = static_cast<int>(v.dims.size());
        for (int i = 0; i < 4; ++i) {
          const int src = i - (4 - rk);
          const int64_t st = (src >= 0 && v.dims[src] != 1) ? v.strides[src] : 0;
          if (st >= (int64_t(1) << 31) || st < 0) return fail(E_UNSUPPORTED_OP, "chain operand stride out of range");
          strides[kx][i] = static_cast<int>(st);
        }
        ptrs[kx] = ptr_of(t, rr);
      }
      Ptr pout = ptr_of(G.out, r);
      // does it fit the open table?
      bool fits = cur.cb.n_req < k::CHAIN_MAX_REQ;
      if (fits && cur.cb.n_req) {
        if (!same_base(pout, cur.out)) fits = false;
        for (int kx = 0; kx <= k::CHAIN_MAX_OPS && fits; ++kx)
          if (opnd[kx] >= 0 && g.tensors[opnd[kx]].kind != TKind::FCONST && !same_base(ptrs[kx], cur.base[kx])) fits = false;
      }
      if (!fits) flush();
      if (!cur.cb.n_req) { cur.out = pout; for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx) cur.base[kx] = ptrs[kx]; }
      k::ChainReq& R = cur.cb.r[cur.cb.n_req++];
      const int oesz = dtype_size(O.dtype);
      for (int i = 0; i < 4; ++i) R.dim[i] = static_cast<int>(od[i]);
      R.out_off = (pout.off - cur.out.off) / oesz;
      bool vec = !red && od[3] % 8 == 0 && R.out_off % 8 == 0 && cur.out.off % 16 == 0;
      for (int kx = 0; kx <= k::CHAIN_MAX_OPS; ++kx) {
        const int t = opnd[kx];
        if (t < 0 || g.tensors[t].kind == TKind::FCONST) continue;
        const int esz = dtype_size(g.tensors[t].dtype);
        R.off[kx] = (ptrs[kx].off - cur.base[kx].off) / esz;
        for (int i = 0; i < 4; ++i) R.stride[kx][i] = strides[kx][i];
        if (strides[kx][3] == 1 || od[3] == 1) {
          // read as 8-element vectors: every address a multiple of 16 bytes (32 for fp32 pairs of float4)
          if (od[3] != 1 && (R.off[kx] % 8 || strides[kx][0] % 8 || strides[kx][1] % 8 || strides[kx][2] % 8 || cur.base[kx].off % 16)) vec = false;
        } else if (strides[kx][3] != 0) vec = false;
      }
      const long long items = red ? od[0] * od[1] * od[2] : (vec && cur.vec ? numel(ov.dims) / 8 : numel(ov.dims));
      if ((red ? items : numel(ov.dims)) >= (int64_t(1) << 31)) return fail(E_UNSUPPORTED_OP, "chain request above 2^31 elements");
      if (!red && cur.vec && !vec) {
        // the table falls back to one element per item: recount the earlier requests
        long long first = 0;
        for (int q = 0; q + 1 < cur.cb.n_req; ++q) {
          cur.cb.r[q].first = first;
          first += static_cast<long long>(cur.cb.r[q].dim[0]) * cur.cb.r[q].dim[1] * cur.cb.r[q].dim[2] * cur.cb.r[q].dim[3];
        }
        cur.cb.total = first;
        cur.vec = false;
      }
      R.first = cur.cb.total;
      cur.cb.total += (!red && !cur.vec) ? numel(ov.dims) : items;
      cur.max_cols = std::max(cur.max_cols, static_cast<int>(od[3]));
      if (od[3] % 16) cur.vec16 = false;
    }
    flush();
    return OK;
  }

  // ------------------------------------------------------------------------------ stand-alone operators (unfused mode)
  Status build_bmm(int gi, const Group& G) {
    const Tensor& A = g.tensors[G.a];
    if (A.dtype != g.tensors[G.w].dtype || A.dtype != g.tensors[G.out].dtype || (A.dtype != DType::BF16 && A.dtype != DType::F32))
      return fail(E_UNSUPPORTED_OP, "MatMul of two activations: operands and result must share one float type");
    for (int r = 0; r < p.n_req; ++r) {
      const View &va = p.views[G.a][r], &vb = p.views[G.w][r], &vc = p.views[G.out][r];
      const int rc = static_cast<int>(vc.dims.size());
      if (rc < 2 || rc > 4 || va.dims.size() < 2 || vb.dims.size() < 2) return fail(E_UNSUPPORTED_OP, "MatMul of two activations supports ranks 2..4");
      if (numel(vc.dims) == 0) continue;
      k::BmmParams bp{};
      bp.is_bf16 = A.dtype == DType::BF16;
      bp.M = static_cast<int>(vc.dims[rc - 2]); bp.N = static_cast<int>(vc.dims[rc - 1]); bp.K = static_cast<int>(va.dims.back());
      bp.B0 = rc >= 4 ? static_cast<int>(vc.dims[0]) : 1;
      bp.B1 = rc >= 3 ? static_cast<int>(vc.dims[rc - 3]) : 1;
      // strides of (b0, b1, row, col) per operand; batch dims right-aligned, extent-1 dims broadcast
      auto fill = [&](const View& v, long long* st) {
        const int rk = static_cast<int>(v.dims.size());
        st[2] = v.strides[rk - 2]; st[3] = v.strides[rk - 1];
        st[1] = (rk >= 3 && v.dims[rk - 3] != 1) ? v.strides[rk - 3] : 0;
        st[0] = (rk >= 4 && v.dims[rk - 4] != 1) ? v.strides[rk - 4] : 0;
      };
      fill(va, bp.as); fill(vb, bp.bs); fill(vc, bp.cs);
      if (vb.dims[vb.dims.size() - 2] != bp.K) return fail(E_SHAPE_CONFLICT, "MatMul inner dims differ");
      Ptr pa = ptr_of(G.a, r), pb = ptr_of(G.w, r), pc = ptr_of(G.out, r);
      add(gi, 1, [=](const RunCtx& x) mutable {
        bp.a = x.resolve(pa); bp.b = x.resolve(pb); bp.c = x.resolve(pc);
        k::bmm_strided<<<dim3((bp.N + 15) / 16, (bp.M + 15) / 16, bp.B0 * bp.B1), 256, 0, x.stream>>>(bp);
        return cudaGetLastError();
      });
    }
    return OK;
  }
  Status build_sumsq(int gi, const Group& G) {
    const Tensor &X = g.tensors[G.a], &O = g.tensors[G.out];
    for (int r = 0; r < p.n_req; ++r) {
      const View &vx = p.views[G.a][r], &vo = p.views[G.out][r];
      if (!vx.contiguous() || !vo.contiguous()) return fail(E_UNSUPPORTED_OP, "ReduceSumSquare needs contiguous operands");
      if (numel(vx.dims) == 0) continue;
      k::SumSqParams sp{};
      sp.D = static_cast<int>(vx.dims.back());
      sp.rows = numel(vx.dims) / sp.D;
      sp.in_bf16 = X.dtype == DType::BF16; sp.out_bf16 = O.dtype == DType::BF16;
      Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r);
      add(gi, 1, [=](const RunCtx& x) mutable {
        sp.x = x.resolve(px); sp.out = x.resolve(po);
        k::reduce_sumsq_rows<<<static_cast<unsigned>((sp.rows + 7) / 8), 256, 0, x.stream>>>(sp);
        return cudaGetLastError();
      });
    }
    return OK;
  }
  Status build_topk_rows(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    if (X.dtype != DType::BF16 && X.dtype != DType::F32) return fail(E_UNSUPPORTED_OP, "TopK ranks float scores");
    for (int r = 0; r < p.n_req; ++r) {
      // either output may be unused by the rest of the graph (then it has no storage)
      const bool has_v = !p.views[G.out].empty(), has_i = !p.views[G.out2].empty();
      if (!has_v && !has_i) continue;
      const View& vx = p.views[G.a][r];
      const View& vk = has_i ? p.views[G.out2][r] : p.views[G.out][r];
      if (!vx.contiguous() || (has_v && !p.views[G.out][r].contiguous()) || (has_i && !p.views[G.out2][r].contiguous()))
        return fail(E_UNSUPPORTED_OP, "TopK needs contiguous operands");
      if (numel(vx.dims) == 0 || numel(vk.dims) == 0) continue;
      k::TopkRowsParams tp{};
      tp.n = static_cast<int>(vx.dims.back());
      tp.k = static_cast<int>(vk.dims.back());
      tp.rows = numel(vx.dims) / tp.n;
      tp.largest = G.act2; tp.by_value = G.act; tp.is_bf16 = X.dtype == DType::BF16;
      if (tp.k > tp.n) return fail(E_BAD_DIM, "TopK: k exceeds the axis length");
      const size_t smem = static_cast<size_t>(tp.n) * 8;
      if (smem > 200 * 1024) return fail(E_UNSUPPORTED_OP, "TopK: axis too long for the shared-memory score table");
      Ptr px = ptr_of(G.a, r), pv = has_v ? ptr_of(G.out, r) : Ptr(), pi = has_i ? ptr_of(G.out2, r) : Ptr();
      add(gi, 1, [=](const RunCtx& x) mutable {
        tp.s = x.resolve(px);
        tp.vals = has_v ? x.resolve(pv) : nullptr;
        tp.idx = has_i ? reinterpret_cast<long long*>(x.resolve(pi)) : nullptr;
        if (smem > 48 * 1024) { static bool once = (cudaFuncSetAttribute(k::topk_rows, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024), true); (void)once; }
        k::topk_rows<<<static_cast<unsigned>(std::min<long long>(tp.rows, 148 * 4)), 256, smem, x.stream>>>(tp);
        return cudaGetLastError();
      });
    }
    return OK;
  }
  Status build_gather(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    for (int r = 0; r < p.n_req; ++r) {
      const View &vx = p.views[G.a][r], &vi = p.views[G.k][r], &vo = p.views[G.out][r];
      if (!vx.contiguous() || !vi.contiguous() || !vo.contiguous()) return fail(E_UNSUPPORTED_OP, "Gather needs contiguous operands");
      if (numel(vo.dims) == 0) continue;
      const int rk = static_cast<int>(vx.dims.size());
      const int ax = G.stride < 0 ? G.stride + rk : G.stride;
      if (ax < 0 || ax >= rk) return fail(E_BAD_DIM, "Gather axis out of range");
      k::GatherParams gp{};
      gp.outer = 1; gp.inner = 1;
      for (int i = 0; i < ax; ++i) gp.outer *= vx.dims[i];
      for (int i = ax + 1; i < rk; ++i) gp.inner *= vx.dims[i];
      gp.n_in = vx.dims[ax];
      gp.n_idx = numel(vi.dims);
      gp.esz = dtype_size(X.dtype);
      if (gp.esz != 2 && gp.esz != 4 && gp.esz != 8) return fail(E_UNSUPPORTED_OP, "Gather element size");
      Ptr px = ptr_of(G.a, r), pi = ptr_of(G.k, r), po = ptr_of(G.out, r);
      const long long total = gp.outer * gp.n_idx * gp.inner;
      add(gi, 1, [=](const RunCtx& x) mutable {
        gp.x = x.resolve(px); gp.idx = reinterpret_cast<const long long*>(x.resolve(pi)); gp.out = x.resolve(po);
        k::gather_axis<<<static_cast<unsigned>(std::max<long long>(1, std::min<long long>((total + 255) / 256, 148 * 16))), 256, 0, x.stream>>>(gp);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  Status build_fill(int gi, const Group& G) {
    const Tensor& O = g.tensors[G.out];
    const Node& n = g.nodes[G.nodes[0]];
    const int dt = O.dtype == DType::I64 ? 2 : O.dtype == DType::BF16 ? 1 : O.dtype == DType::F32 ? 0 : -1;
    if (dt < 0) return fail(E_UNSUPPORTED_OP, "fill: output type");
    for (int r = 0; r < p.n_req; ++r) {
      const View& vo = p.views[G.out][r];
      if (!vo.contiguous()) return fail(E_UNSUPPORTED_OP, "fill: contiguous output");
      if (numel(vo.dims) == 0) continue;
      k::FillParams fp{};
      fp.n = numel(vo.dims);
      fp.dtype = dt;
      if (G.act) {     // Range(start, limit, delta): the value maps hold the operands as expressions of the symbols
        const ValueVal &a = g.tensors[n.ins[0]].V, &d = g.tensors[n.ins[2]].V;
        if (!a.all_known() || !d.all_known() || a.elems.size() != 1 || d.elems.size() != 1) return fail(E_UNSUPPORTED_OP, "Range: start and delta must be known from shapes");
        bool ok1, ok2;
        fp.start = static_cast<double>(e_eval(g.cx, a.elems[0].e, p.b->vals[r], &ok1));
        fp.step = static_cast<double>(e_eval(g.cx, d.elems[0].e, p.b->vals[r], &ok2));
        if (!ok1 || !ok2) return fail(E_UNBOUND_SYMBOL, "Range: operands not bound");
      } else {
        fp.start = G.scale;
        fp.step = 0.0;
      }
      Ptr po = ptr_of(G.out, r);
      add(gi, 1, [=](const RunCtx& x) mutable {
        fp.out = x.resolve(po);
        k::fill_linear<<<static_cast<unsigned>(std::max<long long>(1, std::min<long long>((fp.n + 255) / 256, 148 * 8))), 256, 0, x.stream>>>(fp);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ Resize / Upsample (nearest)
  Status build_resize(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    if (g.tensors[G.out].dtype != X.dtype) return fail(E_UNSUPPORTED_OP, "Resize: output type differs from the input type");
    const int esz = dtype_size(X.dtype);
    if (esz != 2 && esz != 4 && esz != 8) return fail(E_UNSUPPORTED_OP, "Resize: element size");
    for (int r = 0; r < p.n_req; ++r) {
      const View &vx = p.views[G.a][r], &vo = p.views[G.out][r];
      const int rank = static_cast<int>(vo.dims.size());
      if (rank != static_cast<int>(vx.dims.size()) || rank > 6) return fail(E_UNSUPPORTED_OP, "Resize: rank (at most 6, equal to the input's)");
      k::ResizeParams rp{};
      rp.rank = rank;
      rp.esz = esz;
      rp.total = numel(vo.dims);
      if (rp.total == 0) continue;
      if (numel(vx.dims) == 0) return fail(E_BAD_DIM, "Resize: empty input, non-empty output");
      for (int d = 0; d < rank; ++d) {
        rp.in_dim[d] = vx.dims[d]; rp.out_dim[d] = vo.dims[d];
        rp.in_stride[d] = vx.strides[d]; rp.out_stride[d] = vo.strides[d];
        rp.order[d] = rank - 1 - d;
      }
      // walk the output in its storage order: axes by ascending stride
      std::stable_sort(rp.order, rp.order + rank, [&](int a, int b) { return vo.strides[a] < vo.strides[b]; });
      Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r);
      add(gi, 1, [=](const RunCtx& x) mutable {
        rp.x = x.resolve(px);
        rp.out = x.resolve(po);
        const unsigned grid = static_cast<unsigned>(std::max<long long>(1, std::min<long long>((rp.total + 255) / 256, 148 * 16)));
        k::resize_nearest<<<grid, 256, 0, x.stream>>>(rp);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ top-k keep
  Status build_topk(int gi, const Group& G) {
    if (g.tensors[G.a].dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "top-k keep is bf16 only");
    for (int r0 = 0; r0 < p.n_req; r0 += k::COMPACT_MAX_REQ) {
      const int nr = std::min(k::COMPACT_MAX_REQ, p.n_req - r0);
      k::TopkParams tp{};
      tp.n_req = nr;
      Ptr by = ptr_of(G.a, r0), bo = ptr_of(G.out, r0), bi = ptr_of(G.out2, r0);
      int64_t D = -1, total_rows = 0, first_row = 0;
      int nmax = 0;
      for (int i = 0; i < nr; ++i) {
        const int r = r0 + i;
        const View &y = p.views[G.a][r], &o = p.views[G.out][r];
        if (!y.contiguous() || !o.contiguous()) return fail(E_UNSUPPORTED_OP, "top-k keep needs contiguous rows");
        const int64_t d = y.dims.back(), n = numel(y.dims) / d, kk = numel(o.dims) / d;
        if (D < 0) D = d; else if (D != d) return fail(E_UNSUPPORTED_OP, "top-k keep: row length differs");
        if (D % 8) return fail(E_UNSUPPORTED_OP, "top-k keep: rows must be 16-byte multiples");
        Ptr py = ptr_of(G.a, r), po = ptr_of(G.out, r), pi = ptr_of(G.out2, r);
        if (!same_base(py, by) || !same_base(po, bo) || !same_base(pi, bi)) return fail(E_INTERNAL, "top-k bases");
        tp.r[i].row0 = (py.off - by.off) / (D * 2);
        tp.r[i].out_row0 = (po.off - bo.off) / (D * 2);
        tp.r[i].idx0 = (pi.off - bi.off) / 8;
        tp.r[i].n = static_cast<int>(n);
        tp.r[i].k = static_cast<int>(kk);
        if (i == 0) first_row = tp.r[i].row0;
        total_rows = tp.r[i].row0 + n - first_row;
        nmax = std::max(nmax, static_cast<int>(n));
      }
      tp.D = static_cast<int>(D);
      tp.first_row = first_row;
      int chunks = 0;
      for (int i = 0; i < nr; ++i) { tp.chunk_start[i] = chunks; chunks += (tp.r[i].n + k::TOPK_CHUNK - 1) / k::TOPK_CHUNK; }
      tp.chunk_start[nr] = chunks;
      const size_t sc_bytes = (static_cast<size_t>(total_rows) * 8 + 15) & ~size_t(15);
      scratch_need = std::max(scratch_need, sc_bytes + static_cast<size_t>(total_rows));
      const long long rows = total_rows;
      const size_t smem = static_cast<size_t>(nmax) * 8;
      if (smem > 200 * 1024) return fail(E_UNSUPPORTED_OP, "top-k keep: too many tokens per request for the shared-memory score table");
      add(gi, 3, [=](const RunCtx& x) mutable {
        double* score = reinterpret_cast<double*>(x.arena + x.plan->scratch_off[0]);
        tp.y = reinterpret_cast<const __nv_bfloat16*>(x.resolve(by));
        tp.out = reinterpret_cast<__nv_bfloat16*>(x.resolve(bo));
        tp.idx = reinterpret_cast<long long*>(x.resolve(bi));
        tp.score = score;
        tp.keep = reinterpret_cast<unsigned char*>(x.arena + x.plan->scratch_off[0] + sc_bytes);
        // scores are indexed from the first request's first row
        k::ScoreParams sp{tp.y + first_row * tp.D, score, rows, tp.D};
        if (rows) launch_pdl(k::row_sumsq_f64, dim3(static_cast<unsigned>((rows + 7) / 8)), dim3(256), 0, x.stream, sp);
        if (chunks) {
          if (smem > 48 * 1024) cudaFuncSetAttribute(k::topk_flags, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
          launch_pdl(k::topk_flags, dim3(chunks), dim3(256), smem, x.stream, tp);
          launch_pdl(k::topk_gather, dim3(chunks), dim3(256), 0, x.stream, tp);
        }
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ NonZero
  Status build_nonzero(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    if (X.S.rank > 4 || X.S.rank < 1) return fail(E_UNSUPPORTED_OP, "NonZero supports rank 1..4");
    // the runtime symbol that names the count
    const Expr& ce = g.tensors[G.out].S.dims[1].e;
    const int sym = ce.terms.begin()->first[0].first;
    count_known_after(gi, G.out);
    for (int r = 0; r < p.n_req; ++r) {
      const View& v = p.views[G.a][r];
      if (!v.contiguous()) return fail(E_UNSUPPORTED_OP, "NonZero needs a contiguous input");
      k::NonZeroParams np{};
      np.is_bf16 = X.dtype == DType::BF16;
      np.numel = numel(v.dims);
      np.rank = static_cast<int>(v.dims.size());
      for (int i = 0; i < np.rank; ++i) np.dims[i] = v.dims[i];
      np.nblocks = static_cast<int>((np.numel + k::NZ_BLOCK - 1) / k::NZ_BLOCK);
      scratch_need = std::max(scratch_need, static_cast<size_t>(np.nblocks + 1) * 4);
      Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r);
      const size_t count_off = 256 + (static_cast<size_t>(sym) * p.n_req + r) * 8;
      add(gi, 3, [=](const RunCtx& x) mutable {
        np.x = x.resolve(px);
        np.out = reinterpret_cast<long long*>(x.resolve(po));
        np.block_count = reinterpret_cast<int*>(x.arena + x.plan->scratch_off[0]);
        np.count_out = reinterpret_cast<long long*>(x.arena + count_off);
        if (np.nblocks == 0) return cudaMemsetAsync(np.count_out, 0, 8, x.stream);
        k::nonzero_count<<<np.nblocks, k::NZ_BLOCK, 0, x.stream>>>(np);
        k::nonzero_scan<<<1, 1024, 0, x.stream>>>(np);
        k::nonzero_write<<<np.nblocks, k::NZ_BLOCK, 0, x.stream>>>(np);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ layout change
  static bool is_channels_last(const View& v) {
    if (v.dims.size() != 4) return false;
    const int64_t C = v.dims[1], H = v.dims[2], W = v.dims[3];
    return (C == 1 || v.strides[1] == 1) && (W == 1 || v.strides[3] == C) && (H == 1 || v.strides[2] == W * C) &&
           (v.dims[0] == 1 || v.strides[0] == H * W * C);
  }
  Status build_layout(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    const bool from = G.act != 0;
    // requests whose tensors qualify for the vectorised kernels are collected and converted by one launch
    struct Seg { Ptr pi, po; long long HW; int N; };
    std::vector<Seg> segs;
    int segC = -1;
    auto flush = [&]() {
      if (segs.empty()) return;
      std::vector<Seg> batch = segs;
      const int C = segC;
      segs.clear();
      add(gi, 1, [=](const RunCtx& x) {
        k::LayoutBatch B{};
        B.n_seg = static_cast<int>(batch.size());
        B.C = C;
        int tiles = 0;
        bool aligned = true;
        for (int i = 0; i < B.n_seg; ++i) {
          B.in[i] = reinterpret_cast<const __nv_bfloat16*>(x.resolve(batch[i].pi));
          B.out[i] = reinterpret_cast<__nv_bfloat16*>(x.resolve(batch[i].po));
          B.HW[i] = batch[i].HW;
          B.tile_start[i] = tiles;
          tiles += batch[i].N * static_cast<int>((batch[i].HW + 63) / 64);
          aligned = aligned && ((reinterpret_cast<uintptr_t>(B.in[i]) | reinterpret_cast<uintptr_t>(B.out[i])) & 15) == 0;
        }
        B.tile_start[B.n_seg] = tiles;
        if (aligned) {
          const dim3 grid(static_cast<unsigned>(tiles), (C + 63) / 64, 1);
          if (from) k::nhwc_to_nchw_bf16_v8<<<grid, 256, 0, x.stream>>>(B);
          else k::nchw_to_nhwc_bf16_v8<<<grid, 256, 0, x.stream>>>(B);
        } else {   // a caller buffer that is not 16-byte aligned: the element-wise kernels, one tensor at a time
          for (int i = 0; i < B.n_seg; ++i) {
            const dim3 grid(static_cast<unsigned>((B.HW[i] + 63) / 64), (C + 63) / 64, batch[i].N);
            if (from) k::nhwc_to_nchw_bf16<<<grid, 256, 0, x.stream>>>(B.in[i], B.out[i], C, B.HW[i]);
            else k::nchw_to_nhwc_bf16<<<grid, 256, 0, x.stream>>>(B.in[i], B.out[i], C, B.HW[i]);
          }
        }
        return cudaGetLastError();
      });
    };
    for (int r = 0; r < p.n_req; ++r) {
      const View &vi = p.views[G.a][r], &vo = p.views[G.out][r];
      const int64_t n = numel(vi.dims);
      if (!n) continue;
      Ptr pi = ptr_of(G.a, r), po = ptr_of(G.out, r);
      const bool spatial = vi.dims.size() == 4 && vi.dims[2] * vi.dims[3] > 1 && vi.dims[1] > 1;
      if (!spatial) {  // both layouts coincide: plain copy
        const size_t bytes = static_cast<size_t>(n) * dtype_size(X.dtype);
        add(gi, 1, [=](const RunCtx& x) { return cudaMemcpyAsync(x.resolve(po), x.resolve(pi), bytes, cudaMemcpyDeviceToDevice, x.stream); });
        continue;
      }
      if (X.dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "layout change is bf16 only");
      const View& nchw = G.act ? vo : vi;
      const View& cl = G.act ? vi : vo;
      if (!nchw.contiguous() || !is_channels_last(cl)) return fail(E_UNSUPPORTED_OP, "layout change between unexpected layouts");
      const int N = static_cast<int>(vi.dims[0]), C = static_cast<int>(vi.dims[1]);
      const long long HW = vi.dims[2] * vi.dims[3];
      if (C % 8 == 0 && HW % 8 == 0 && N * ((HW + 63) / 64) < (1ll << 28)) {
        if (segC >= 0 && segC != C) flush();
        segC = C;
        segs.push_back(Seg{pi, po, HW, N});
        if (segs.size() == static_cast<size_t>(k::LAYOUT_MAX_SEG)) flush();
        continue;
      }
      add(gi, 1, [=](const RunCtx& x) {
        const dim3 grid(static_cast<unsigned>((HW + 63) / 64), (C + 63) / 64, N);
        auto* in = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pi));
        auto* out = reinterpret_cast<__nv_bfloat16*>(x.resolve(po));
        if (from) k::nhwc_to_nchw_bf16<<<grid, 256, 0, x.stream>>>(in, out, C, HW);
        else k::nchw_to_nhwc_bf16<<<grid, 256, 0, x.stream>>>(in, out, C, HW);
        return cudaGetLastError();
      });
    }
    flush();
    return OK;
  }

  // ------------------------------------------------------------------------------ thin-channel convolution
  // (e.g. the RGB stem): patches are gathered into an [pixels, Kp] matrix in scratch, then the GEMM
  // kernel runs with the fused bias / activation epilogue; its [pixels, Cout] output is channels-last.
  Status build_conv_im2col(int gi, const Group& G) {
    const Tensor& W = g.tensors[G.w];
    const int Cout = static_cast<int>(W.S.dims[0].e.const_value()), Cin = static_cast<int>(W.S.dims[1].e.const_value());
    const int ks = static_cast<int>(W.S.dims[2].e.const_value());
    if (G.res >= 0 || G.act2 || G.has_ln) return fail(E_UNSUPPORTED_OP, "thin-channel convolution: unsupported epilogue tail");
    if (Cout % 8) return fail(E_UNSUPPORTED_OP, "thin-channel convolution needs Cout % 8 == 0");
    size_t pk = 0;
    for (size_t i = 0; i < c.packed_consts.size(); ++i) if (c.packed_consts[i] == G.w) pk = c.packed_off[i];
    if (is_fused_stem(c, G)) {
      for (int r = 0; r < p.n_req; ++r) {
        const View &vx = p.views[G.a][r], &vo = p.views[G.out][r];
        if (!numel(vo.dims)) continue;
        if (!vx.contiguous()) return fail(E_UNSUPPORTED_OP, "thin-channel convolution reads an NCHW-contiguous input");
        if (!is_channels_last(vo)) return fail(E_UNSUPPORTED_OP, "convolution output must be stored channels-last");
        k::StemParams sp{};
        sp.N = static_cast<int>(vx.dims[0]); sp.H = static_cast<int>(vx.dims[2]); sp.W = static_cast<int>(vx.dims[3]);
        sp.Ho = static_cast<int>(vo.dims[2]); sp.Wo = static_cast<int>(vo.dims[3]);
        Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r), pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
        Ptr pw; pw.where = 5; pw.off = static_cast<int64_t>(pk);
        const bool hb = G.bias >= 0;
        const int act = G.act;
        struct Cache { const void* w = nullptr; const void* o = nullptr; const void* xin = nullptr; CUtensorMap tw, to, tx; };
        auto cache = std::make_shared<Cache>();
        add(gi, 1, [=](const RunCtx& x) mutable {
          sp.x = reinterpret_cast<const __nv_bfloat16*>(x.resolve(px));
          sp.bias = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
          sp.vec_ok = (reinterpret_cast<uintptr_t>(sp.x) % 16 == 0 && sp.W % 8 == 0) ? 1 : 0;
          sp.status = reinterpret_cast<int*>(x.arena);
          const void* Wp = x.resolve(pw);
          void* O = x.resolve(po);
          if (cache->w != Wp || cache->o != O || cache->xin != sp.x) {
            if (!encode_bf16_kchunks(&cache->tw, Wp, 64, 192, 192, 64, 3) ||
                !encode_bf16_nhwc(&cache->to, O, static_cast<uint64_t>(sp.N), static_cast<uint64_t>(sp.Ho), static_cast<uint64_t>(sp.Wo), 64, 128, 1, 1))
              return cudaErrorInvalidValue;
            // input patches by TMA where the rows are 16-byte multiples; otherwise the builder warps copy them
            if (sp.vec_ok && !encode_bf16_planes(&cache->tx, sp.x, static_cast<uint64_t>(sp.N) * 3, static_cast<uint64_t>(sp.H), static_cast<uint64_t>(sp.W), k::STEM_BOX_W, 7))
              return cudaErrorInvalidValue;
            if (!sp.vec_ok) cache->tx = cache->tw;      // unused by that variant
            cache->w = Wp; cache->o = O; cache->xin = sp.x;
          }
          const long long tiles = static_cast<long long>(sp.N) * sp.Ho * ((sp.Wo + 127) / 128);
          if (tiles >= (1ll << 31)) return cudaErrorInvalidValue;
          const dim3 gd(static_cast<unsigned>(std::min<long long>(tiles, x.plan->sm_count))), bd(k::STEM_THREADS);
#define SOD2_STEM_CASE(ACT_, TMA_)                                                                                            \
          {                                                                                                                  \
            static bool once = (cudaFuncSetAttribute(k::conv_stem_bf16_tcgen05<ACT_, TMA_>, cudaFuncAttributeMaxDynamicSharedMemorySize, k::STEM_SMEM), true); \
            (void)once;                                                                                                      \
            launch_pdl(k::conv_stem_bf16_tcgen05<ACT_, TMA_>, gd, bd, k::STEM_SMEM, x.stream, cache->tw, cache->to, cache->tx, sp);  \
          }
          if (act == 2) { if (sp.vec_ok) SOD2_STEM_CASE(2, true) else SOD2_STEM_CASE(2, false) }
          else { if (sp.vec_ok) SOD2_STEM_CASE(0, true) else SOD2_STEM_CASE(0, false) }
#undef SOD2_STEM_CASE
          return cudaGetLastError();
        });
      }
      return OK;
    }
    const int K = Cin * ks * ks, Kp = (K + 63) / 64 * 64;
    for (int r = 0; r < p.n_req; ++r) {
      const View &vx = p.views[G.a][r], &vo = p.views[G.out][r];
      if (!numel(vo.dims)) continue;
      if (!vx.contiguous()) return fail(E_UNSUPPORTED_OP, "thin-channel convolution reads an NCHW-contiguous input");
      if (!is_channels_last(vo)) return fail(E_UNSUPPORTED_OP, "convolution output must be stored channels-last");
      k::Im2colParams ip{};
      ip.N = static_cast<int>(vx.dims[0]); ip.C = Cin; ip.H = static_cast<int>(vx.dims[2]); ip.W = static_cast<int>(vx.dims[3]);
      ip.Ho = static_cast<int>(vo.dims[2]); ip.Wo = static_cast<int>(vo.dims[3]);
      ip.ks = ks; ip.stride = G.stride; ip.pad = G.pad; ip.K = K; ip.Kp = Kp;
      const long long M = static_cast<long long>(ip.N) * ip.Ho * ip.Wo;
      scratch_need = std::max(scratch_need, static_cast<size_t>(M) * Kp * 2);
      Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r), pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
      Ptr pw; pw.where = 5; pw.off = static_cast<int64_t>(pk);
      const bool hb = G.bias >= 0;
      const int act = G.act;
      struct Cache { const void* a = nullptr; const void* w = nullptr; const void* o = nullptr; CUtensorMap ta, tb, to; };
      auto cache = std::make_shared<Cache>();
      add(gi, 2, [=](const RunCtx& x) mutable {
        ip.x = reinterpret_cast<const __nv_bfloat16*>(x.resolve(px));
        ip.a = reinterpret_cast<__nv_bfloat16*>(x.arena + x.plan->scratch_off[0]);
        {
          const int segs = (ip.Wo + 63) / 64;
          const size_t wsm = ((static_cast<size_t>(ip.C) * ip.ks * (63 * ip.stride + ip.ks) + 7) & ~size_t(7)) * 2 + static_cast<size_t>(ip.Kp) * 4;
          k::im2col_nchw_bf16<<<static_cast<unsigned>(segs) * ip.Ho * ip.N, 256, wsm, x.stream>>>(ip);
        }
        const void* Wp = x.resolve(pw);
        void* O = x.resolve(po);
        if (cache->a != ip.a || cache->w != Wp || cache->o != O) {
          if (!encode_bf16_kchunks(&cache->ta, ip.a, M, Kp, Kp, 128, 2) || !encode_bf16_kchunks(&cache->tb, Wp, Cout, Kp, Kp, 128, 2) ||
              !encode_bf16_2d(&cache->to, O, M, Cout, Cout, 128))
            return cudaErrorInvalidValue;
          cache->a = ip.a; cache->w = Wp; cache->o = O;
        }
        k::GemmEpilogue ep{};
        ep.bias = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
        ep.status = reinterpret_cast<int*>(x.arena);
        const long long tiles = ((M + 127) / 128) * ((Cout + 127) / 128);
        const dim3 gd(static_cast<unsigned>(std::min<long long>(tiles, x.plan->sm_count))), bd(k::GEMM_THREADS);
        constexpr int smem = k::GemmSmem<128, 2, 3>::TOTAL;
        if (act == 2) {
          cudaFuncSetAttribute(k::gemm_bf16_tcgen05<128, 2, 3, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
          launch_pdl(k::gemm_bf16_tcgen05<128, 2, 3, 2>, gd, bd, smem, x.stream, cache->ta, cache->tb, cache->to, cache->to, static_cast<int>(M), Cout, Kp, ep);
        } else {
          cudaFuncSetAttribute(k::gemm_bf16_tcgen05<128, 2, 3, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
          launch_pdl(k::gemm_bf16_tcgen05<128, 2, 3, 0>, gd, bd, smem, x.stream, cache->ta, cache->tb, cache->to, cache->to, static_cast<int>(M), Cout, Kp, ep);
        }
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ convolution
  Status build_conv(int gi, const Group& G) {
    const Tensor& W = g.tensors[G.w];
    if (W.dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "convolution is bf16 only");
    const int Cout = static_cast<int>(W.S.dims[0].e.const_value()), Cin = static_cast<int>(W.S.dims[1].e.const_value());
    const int ks = static_cast<int>(W.S.dims[2].e.const_value());
    if (W.S.dims[3].e.const_value() != ks) return fail(E_UNSUPPORTED_OP, "convolution needs a square kernel");
    if (Cin % 64) return build_conv_im2col(gi, G);
    if (Cout % 64) return fail(E_UNSUPPORTED_OP, "implicit-GEMM convolution needs Cout % 64 == 0");
    if (G.has_ln || (G.act != 0 && G.act != 2)) return fail(E_UNSUPPORTED_OP, "convolution epilogue: unsupported tail");
    size_t pk = 0;
    for (size_t i = 0; i < c.packed_consts.size(); ++i) if (c.packed_consts[i] == G.w) pk = c.packed_off[i];
    const int bn = (Cout % 128 == 0) ? 128 : 64;
    const int kch = 2;
    // the table of per-sample channel sums this convolution adds its outputs to (the last convolution of an
    // in-place gated block), or SIZE_MAX
    const size_t gap_table = gap_accum.count(gi) ? gap_accum[gi] : SIZE_MAX;
    // requests that take the row-halo kernel are collected and launched together (up to C3_MAX_REQ per launch)
    struct RowsReq { Ptr px, po, pr; int H, W, Ho, Wo, n_img, n_in_map, n_out_map, n_res_map; k::ConvParams cp; bool rt; size_t rt_slot; long long ids_in, ids_res, ids_out; };
    std::vector<RowsReq> rows_reqs;
    Ptr pw_all; pw_all.where = 5; pw_all.off = static_cast<int64_t>(pk);
    Ptr pb_all = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
    auto emit_rows = [&](std::vector<RowsReq> batch) {
      const bool hb = G.bias >= 0, hr = G.res >= 0;
      const int act = G.act;
      const bool wres = Cin == 64 && Cout == 64;
      const int K = 9 * Cin;
      const Ptr pw = pw_all, pb = pb_all;
      struct Cache { std::vector<const void*> key; CUtensorMap tw; k::Conv3Batch B; };
      auto cache = std::make_shared<Cache>();
      long long tiles = 0;
      for (auto& q : batch) tiles += static_cast<long long>((q.Wo + 127) / 128) * q.Ho * q.n_img;
      tiles *= (Cout + bn - 1) / bn;
      add(gi, 1, [=](const RunCtx& x) mutable {
        std::vector<const void*> key;
        const void* Wp = x.resolve(pw);
        key.push_back(Wp);
        for (auto& q : batch) { key.push_back(x.resolve(q.px)); key.push_back(x.resolve(q.po)); key.push_back(hr ? x.resolve(q.pr) : nullptr); }
        if (cache->key != key) {
          k::Conv3Batch& B = cache->B;
          B.n_req = static_cast<int>(batch.size());
          int ts = 0;
          for (size_t i = 0; i < batch.size(); ++i) {
            const RowsReq& q = batch[i];
            const void* X = key[1 + 3 * i];
            void* O = const_cast<void*>(key[2 + 3 * i]);
            const void* R = hr ? key[3 + 3 * i] : O;
            if (!encode_bf16_nhwc(&B.tx[i], X, q.n_in_map, q.H, q.W, Cin, 130, 1, 1) ||
                !encode_bf16_nhwc(&B.to[i], O, q.n_out_map, q.Ho, q.Wo, Cout, 128, 1, 1) ||
                !encode_bf16_nhwc(&B.tr[i], R, hr ? q.n_res_map : q.n_out_map, q.Ho, q.Wo, Cout, 128, 1, 1))
              return cudaErrorInvalidValue;
            B.tile_start[i] = ts;
            ts += ((q.Wo + 127) / 128) * q.Ho * q.n_img;
            B.Ho[i] = q.Ho; B.Wo[i] = q.Wo;
          }
          B.tile_start[batch.size()] = ts;
          if (!encode_bf16_kchunks(&cache->tw, Wp, Cout, K, K, bn, 3)) return cudaErrorInvalidValue;
          cache->key = key;
        }
        k::ConvParams cp = batch[0].cp;
        cp.bias = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
        cp.status = reinterpret_cast<int*>(x.arena);
        cp.n_img_ptr = batch[0].rt ? reinterpret_cast<const long long*>(x.arena + batch[0].rt_slot) : nullptr;
        const char* auxb = x.arena + x.plan->scratch_off[1];
        cp.in_ids = batch[0].ids_in >= 0 ? reinterpret_cast<const int*>(auxb + batch[0].ids_in) : nullptr;
        cp.res_ids = batch[0].ids_res >= 0 ? reinterpret_cast<const int*>(auxb + batch[0].ids_res) : nullptr;
        cp.out_ids = batch[0].ids_out >= 0 ? reinterpret_cast<const int*>(auxb + batch[0].ids_out) : nullptr;
        cp.gap_sum = (gap_table != SIZE_MAX && batch.size() == 1) ? reinterpret_cast<double*>(const_cast<char*>(auxb) + gap_table) : nullptr;
        const dim3 gd(static_cast<unsigned>(std::min<long long>(tiles, x.plan->sm_count)));
        const int variant = ((wres ? 4 : 0) + (bn == 128 ? 2 : 0) + (act == 2 ? 1 : 0)) * 2 + (hr ? 1 : 0);
#define SOD2_CONV3_CASE(V, BN_, RES_, ST_, ACT_, HR_)                                                                    \
        case V: {                                                                                                        \
          constexpr int smem = k::Conv3Smem<BN_, RES_, ST_>::TOTAL;                                                       \
          static bool once = (cudaFuncSetAttribute(k::conv3x3_rows_bf16_tcgen05<BN_, RES_, ST_, ACT_, HR_>,               \
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);             \
          (void)once;                                                                                                    \
          launch_pdl(k::conv3x3_rows_bf16_tcgen05<BN_, RES_, ST_, ACT_, HR_>, gd, dim3(k::CONV3_THREADS), smem, x.stream, cache->B, cache->tw, cp); \
        } break;
        switch (variant) {
          SOD2_CONV3_CASE(0, 64, false, 4, 0, false)
          SOD2_CONV3_CASE(1, 64, false, 4, 0, true)
          SOD2_CONV3_CASE(2, 64, false, 4, 2, false)
          SOD2_CONV3_CASE(3, 64, false, 4, 2, true)
          SOD2_CONV3_CASE(4, 128, false, 3, 0, false)
          SOD2_CONV3_CASE(5, 128, false, 3, 0, true)
          SOD2_CONV3_CASE(6, 128, false, 3, 2, false)
          SOD2_CONV3_CASE(7, 128, false, 3, 2, true)
          SOD2_CONV3_CASE(8, 64, true, 7, 0, false)
          SOD2_CONV3_CASE(9, 64, true, 7, 0, true)
          SOD2_CONV3_CASE(10, 64, true, 7, 2, false)
          default:
          SOD2_CONV3_CASE(11, 64, true, 7, 2, true)
        }
#undef SOD2_CONV3_CASE
        return cudaGetLastError();
      });
    };
    for (int r = 0; r < p.n_req; ++r) {
      const View &vx = p.views[G.a][r], &vo = p.views[G.out][r];
      if (!numel(vo.dims) || !numel(vx.dims)) continue;
      if (!is_channels_last(vx) || !is_channels_last(vo)) return fail(E_UNSUPPORTED_OP, "convolution operands must be stored channels-last");
      if (G.res >= 0 && !is_channels_last(p.views[G.res][r])) return fail(E_UNSUPPORTED_OP, "convolution residual must be stored channels-last");
      if (vx.dims[1] != Cin || vo.dims[1] != Cout) return fail(E_SHAPE_CONFLICT, "convolution channel counts");
      k::ConvParams cp{};
      cp.n_img = static_cast<int>(vo.dims[0]);
      cp.Ho = static_cast<int>(vo.dims[2]); cp.Wo = static_cast<int>(vo.dims[3]);
      cp.Cin = Cin; cp.Cout = Cout; cp.ksize = ks; cp.stride = G.stride; cp.pad = G.pad;
      cp.korder = ks == 3;
      cp.has_residual = G.res >= 0;
      cp.act2 = G.act2;
      const RtCount rc = runtime_count(G.out, r);
      cp.cnt_a = rc.a; cp.cnt_b = rc.b;
      const bool rt = rc.rt;
      const size_t rt_slot = rc.slot_off;
      // index-indirect operands: offsets of their id lists in the Switch groups' index area
      long long ids_in = -1, ids_res = -1, ids_out = -1;
      {
        auto ids_of = [&](int t, long long* off) -> bool {
          const View& v = p.views[t][r];
          if (v.ind_gate < 0) return true;
          auto it = switch_aux.find(v.ind_gate);
          if (it == switch_aux.end()) return false;
          const int Nall = static_cast<int>(p.views[p.root_of[t]][r].dims[0]);
          *off = static_cast<long long>(it->second) + (v.ind_list ? static_cast<long long>(Nall) * 4 : 0);
          return true;
        };
        if (!ids_of(G.a, &ids_in) || !ids_of(G.out, &ids_out) || (G.res >= 0 && !ids_of(G.res, &ids_res)))
          return fail(E_INTERNAL, "index-indirect convolution operand without a Switch");
      }
      // pixel patch of a tile: the 128-pixel shape that wastes the fewest padded pixels
      long long best = -1;
      for (int tw : {128, 64, 32, 16, 8}) {
        const int th = 128 / tw;
        const long long padded = static_cast<long long>((cp.Wo + tw - 1) / tw) * tw * ((cp.Ho + th - 1) / th) * th;
        if (best < 0 || padded < best) { best = padded; cp.TW = tw; cp.TH = th; }
      }
      // wide images with a 3x3 / stride 1 / pad 1 kernel: row-halo kernel (a tile is 128 pixels of one row)
      const bool rows = ks == 3 && G.stride == 1 && G.pad == 1 && cp.Wo >= 96 && ((cp.Wo + 127) / 128) * 128 * 4 <= cp.Wo * 5;
      if (rows) { cp.TW = 128; cp.TH = 1; }
      if (cp.TW * G.stride > 256 || cp.TH * G.stride > 256) return fail(E_UNSUPPORTED_OP, "convolution stride too large for the TMA box");
      const int H = static_cast<int>(vx.dims[2]), Wd = static_cast<int>(vx.dims[3]);
      Ptr px = ptr_of(G.a, r), po = ptr_of(G.out, r), pr = G.res >= 0 ? ptr_of(G.res, r) : Ptr();
      Ptr pw; pw.where = 5; pw.off = static_cast<int64_t>(pk);
      Ptr pb = G.bias >= 0 ? ptr_of(G.bias, 0) : Ptr();
      const bool hb = G.bias >= 0, hr = G.res >= 0;
      const int act = G.act, stride = G.stride;
      const int K = ks * ks * Cin;
      const long long tiles = static_cast<long long>((cp.Wo + cp.TW - 1) / cp.TW) * ((cp.Ho + cp.TH - 1) / cp.TH) * cp.n_img * ((Cout + bn - 1) / bn);
      // images covered by each operand's tensor map: all images of the root for an index-indirect operand
      const int n_in_map = static_cast<int>(vx.ind_gate >= 0 ? p.views[p.root_of[G.a]][r].dims[0] : vx.dims[0]);
      const int n_out_map = static_cast<int>(vo.ind_gate >= 0 ? p.views[p.root_of[G.out]][r].dims[0] : vo.dims[0]);
      const int n_res_map = G.res >= 0 ? static_cast<int>(p.views[G.res][r].ind_gate >= 0 ? p.views[p.root_of[G.res]][r].dims[0] : p.views[G.res][r].dims[0]) : 0;
      if (rows) {
        RowsReq q{px, po, pr, H, Wd, cp.Ho, cp.Wo, cp.n_img, n_in_map, n_out_map, n_res_map, cp, rt, rt_slot, ids_in, ids_res, ids_out};
        // a run-time image count or id lists belong to one request: such a request is launched alone
        const bool solo = rt || ids_in >= 0 || ids_res >= 0 || ids_out >= 0;
        if (solo) { emit_rows({q}); continue; }
        rows_reqs.push_back(q);
        if (rows_reqs.size() == static_cast<size_t>(k::C3_MAX_REQ)) { emit_rows(rows_reqs); rows_reqs.clear(); }
        continue;
      }
      struct Cache { const void* a = nullptr; const void* w = nullptr; const void* o = nullptr; const void* r = nullptr; CUtensorMap tx, tw, to, tr; };
      auto cache = std::make_shared<Cache>();
      add(gi, 1, [=](const RunCtx& x) mutable {
        const void* X = x.resolve(px);
        const void* Wp = x.resolve(pw);
        void* O = x.resolve(po);
        const void* R = hr ? x.resolve(pr) : O;
        if (cache->a != X || cache->w != Wp || cache->o != O || cache->r != R) {
          if (!encode_bf16_nhwc(&cache->tx, X, n_in_map, H, Wd, Cin, cp.TW, cp.TH, stride) ||
              !encode_bf16_kchunks(&cache->tw, Wp, Cout, K, K, bn, kch) ||
              !encode_bf16_nhwc(&cache->to, O, n_out_map, cp.Ho, cp.Wo, Cout, cp.TW, cp.TH, 1) ||
              !encode_bf16_nhwc(&cache->tr, R, hr ? n_res_map : n_out_map, cp.Ho, cp.Wo, Cout, cp.TW, cp.TH, 1))
            return cudaErrorInvalidValue;
          cache->a = X; cache->w = Wp; cache->o = O; cache->r = R;
        }
        cp.bias = hb ? reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb)) : nullptr;
        cp.status = reinterpret_cast<int*>(x.arena);
        cp.n_img_ptr = rt ? reinterpret_cast<const long long*>(x.arena + rt_slot) : nullptr;
        const char* auxb = x.arena + x.plan->scratch_off[1];
        cp.in_ids = ids_in >= 0 ? reinterpret_cast<const int*>(auxb + ids_in) : nullptr;
        cp.res_ids = ids_res >= 0 ? reinterpret_cast<const int*>(auxb + ids_res) : nullptr;
        cp.out_ids = ids_out >= 0 ? reinterpret_cast<const int*>(auxb + ids_out) : nullptr;
        cp.gap_sum = gap_table != SIZE_MAX ? reinterpret_cast<double*>(const_cast<char*>(auxb) + gap_table) : nullptr;
        const dim3 gd(static_cast<unsigned>(std::min<long long>(tiles, x.plan->sm_count))), bd(k::CONV_THREADS);
        const int variant = ((bn == 128 ? 2 : 0) + (act == 2 ? 1 : 0)) * 2 + (hr ? 1 : 0);
#define SOD2_CONV_CASE(V, BN_, KCH_, ST_, ACT_, HR_)                                                                     \
        case V: {                                                                                                        \
          constexpr int smem = k::ConvSmem<BN_, KCH_, ST_>::TOTAL;                                                        \
          static bool once = (cudaFuncSetAttribute(k::conv_igemm_bf16_tcgen05<BN_, KCH_, ST_, ACT_, HR_>,                 \
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, smem), true);             \
          (void)once;                                                                                                    \
          launch_pdl(k::conv_igemm_bf16_tcgen05<BN_, KCH_, ST_, ACT_, HR_>, gd, bd, smem, x.stream, cache->tx, cache->tw, \
                     cache->to, cache->tr, cp);                                                                          \
        } break;
        switch (variant) {
          SOD2_CONV_CASE(0, 64, 2, 4, 0, false)
          SOD2_CONV_CASE(1, 64, 2, 4, 0, true)
          SOD2_CONV_CASE(2, 64, 2, 4, 2, false)
          SOD2_CONV_CASE(3, 64, 2, 4, 2, true)
          SOD2_CONV_CASE(4, 128, 2, 3, 0, false)
          SOD2_CONV_CASE(5, 128, 2, 3, 0, true)
          SOD2_CONV_CASE(6, 128, 2, 3, 2, false)
          default:
          SOD2_CONV_CASE(7, 128, 2, 3, 2, true)
        }
#undef SOD2_CONV_CASE
        return cudaGetLastError();
      });
    }
    if (!rows_reqs.empty()) emit_rows(rows_reqs);
    return OK;
  }

  // ------------------------------------------------------------------------------ run-time sample counts
  // A tensor whose leading extent is execution determined (gated sub-batch): extent = a + b * count,
  // where count is the run-time symbol's slot in the arena header, written by the Switch group.
  int rt_symbol_of(int t) const {
    const ShapeVal& sv = g.tensors[t].S;
    for (const Dim& d : sv.dims)
      if (d.known())
        for (auto& term : d.e.terms)
          for (auto& pw : term.first)
            if (g.cx.atoms[pw.first].kind == AtomKind::SYM && g.cx.atoms[pw.first].runtime) return pw.first;
    return -1;
  }
  void count_known_after(int gi, int tensor) {
    if (p.rt_syms_after.size() != c.groups.size()) p.rt_syms_after.assign(c.groups.size(), {});
    const int sym = rt_symbol_of(tensor);
    if (sym >= 0) p.rt_syms_after[gi].push_back(sym);
  }
  struct RtCount { bool rt = false; size_t slot_off = 0; int a = 0, b = 0; };
  RtCount runtime_count(int t, int r) const {
    RtCount rc;
    const ShapeVal& s = g.tensors[t].S;
    if (s.rank < 1 || !s.dims[0].known() || !e_has_runtime(g.cx, s.dims[0].e)) return rc;
    int sym = -1;
    for (auto& term : s.dims[0].e.terms)
      for (auto& pw : term.first)
        if (g.cx.atoms[pw.first].kind == AtomKind::SYM && g.cx.atoms[pw.first].runtime) sym = pw.first;
    if (sym < 0) return rc;
    std::vector<int64_t> vals = p.b->vals[r];
    bool ok0, ok1;
    vals[sym] = 0;
    const int64_t v0 = e_eval(g.cx, s.dims[0].e, vals, &ok0);
    vals[sym] = 1;
    const int64_t v1 = e_eval(g.cx, s.dims[0].e, vals, &ok1);
    if (!ok0 || !ok1) return rc;
    rc.rt = true;
    rc.slot_off = 256 + (static_cast<size_t>(sym) * p.n_req + r) * 8;
    rc.a = static_cast<int>(v0);
    rc.b = static_cast<int>(v1 - v0);
    return rc;
  }
  // persistent side storage of a Switch (index lists), found again by the Combine through the gate tensor
  std::map<int, size_t> switch_aux;   // gate tensor -> offset inside the aux region
  size_t aux_need = 0;
  std::set<int> partition_fused;      // gate tensors whose id partition is computed by the gate kernel
  int n_tickets = 0;
  // Per-sample channel sums carried from gate to gate (aux region): `gapsum_root` is the storage root whose
  // current contents the table at `gapsum_aux` describes.  A gate on that storage skips the pooling pass; the
  // last convolution of an in-place block (group index in gap_accum) adds the executed samples' new sums.
  int gapsum_root = -1;
  size_t gapsum_aux = 0;
  std::map<int, size_t> gap_accum;    // convolution group -> offset of the table it accumulates into

  // ------------------------------------------------------------------------------ gate (decision scalar)
  Status build_gate(int gi, const Group& G) {
    if (g.tensors[G.a].dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "gate is bf16 only");
    const bool want_z = std::find(G.ext_out.begin(), G.ext_out.end(), G.out2) != G.ext_out.end();
    for (int r = 0; r < p.n_req; ++r) {
      const View& vx = p.views[G.a][r];
      if (!numel(vx.dims)) continue;
      if (!is_channels_last(vx)) return fail(E_UNSUPPORTED_OP, "gate reads channels-last storage");
      k::GapParams gp{};
      gp.C = static_cast<int>(vx.dims[1]);
      gp.HW = vx.dims[2] * vx.dims[3];
      const int N = static_cast<int>(vx.dims[0]);
      // N images x slabs CTAs: about four per SM, each with enough pixels to keep loads in flight
      gp.slabs = static_cast<int>(std::max<long long>(1, std::min<long long>(std::max(1, 592 / N), gp.HW / 16)));
      scratch_need = std::max(scratch_need, static_cast<size_t>(N) * gp.slabs * gp.C * 8);
      Ptr px = ptr_of(G.a, r), pw = ptr_of(G.w, 0), pb = ptr_of(G.bias, 0), pg = ptr_of(G.out, r);
      Ptr pz = want_z ? ptr_of(G.out2, r) : Ptr();
      const bool zb = want_z && g.tensors[G.out2].dtype == DType::BF16;
      // The Switch that regroups the samples by this gate needs the stable partition of the sample ids.
      // The last CTA of the logit kernel computes it (ticket counters live in bytes 128.. of the arena
      // header, which every run clears), so the Switch launches nothing of its own for it.
      bool fuse_part = false;
      size_t part_aux = 0, part_slot = 0;
      const int ticket = n_tickets;
      if (p.n_req == 1 && ticket < 32) {
        for (const Group& S : c.groups) {
          if (S.kind != GKind::SWITCH || S.gate != G.out || switch_aux.count(S.gate)) continue;
          RtCount rc = runtime_count(S.out, 0);
          if (!rc.rt || rc.a != 0 || rc.b != 1) break;
          part_aux = aux_need;
          switch_aux[S.gate] = part_aux;
          aux_need += (static_cast<size_t>(2 * N) * 4 + 16 + 255) & ~size_t(255);
          part_slot = rc.slot_off;
          partition_fused.insert(S.gate);
          count_known_after(gi, S.out);
          fuse_part = true;
          ++n_tickets;
          break;
        }
      }
      // Per-sample channel sums: reuse the table if it describes this tensor's storage, else pool (two
      // launches) into a new table.  If the block is an in-place, index-indirect one, its last convolution
      // accumulates the executed samples' sums into the table and the next gate finds it up to date.
      const int xroot = p.root_of[G.a];
      const bool whole = vx.offset == 0 && vx.ind_gate < 0;
      const bool have_sums = fuse_part && whole && gapsum_root >= 0 && gapsum_root == xroot;
      size_t table = gapsum_aux;
      bool keep_table = false;
      if (fuse_part && whole) {
        if (!have_sums) { table = aux_need; aux_need += (static_cast<size_t>(N) * gp.C * 8 + 255) & ~size_t(255); }
        // look ahead: Switch on this gate -> index-indirect -> Combine whose output lives in this storage -> its writer
        int writer = -1;
        bool in_place = false;          // the block overwrites this storage
        for (size_t ci = 0; ci < c.groups.size() && writer < 0; ++ci) {
          const Group& Cb = c.groups[ci];
          if (Cb.kind != GKind::COMBINE || Cb.gate != G.out || c.storage[Cb.out].kind != Storage::ALIAS) continue;
          if (p.views[Cb.out].empty() || p.root_of[Cb.out] != xroot) continue;
          in_place = true;
          for (size_t wi = 0; wi < c.groups.size(); ++wi) {
            const Group& Wg = c.groups[wi];
            if (Wg.kind == GKind::CONV && Wg.out >= 0 && c.storage[Wg.out].kind == Storage::INDIRECT_OUT && c.storage[Wg.out].other == Cb.out &&
                g.tensors[Wg.w].S.dims[1].e.const_value() % 64 == 0) { writer = static_cast<int>(wi); break; }
          }
        }
        // accumulating in the convolution's epilogue costs about as much per byte as the pooling pass it
        // replaces; what it saves is the pass's two launches, which only outweighs it on the smaller tensors
        if (writer >= 0 && static_cast<double>(N) * gp.C * static_cast<double>(gp.HW) * 2.0 > 32e6) writer = -1;
        if (writer >= 0) { gap_accum[writer] = table; keep_table = true; }
        gapsum_root = (in_place && writer < 0) ? -1 : xroot;   // overwritten without the sums being kept: the table goes stale
        gapsum_aux = table;
      }
      const bool zero_exec = keep_table;
      const bool pool = !have_sums;
      const bool to_table = fuse_part && whole;     // sums go to the aux table (else: slab partials in scratch, as before)
      add(gi, pool ? (to_table ? 3 : 2) : 1, [=](const RunCtx& x) mutable {
        char* auxb = x.arena + x.plan->scratch_off[1];
        double* sums = reinterpret_cast<double*>(auxb + table);
        gp.x = reinterpret_cast<const __nv_bfloat16*>(x.resolve(px));
        gp.partial = reinterpret_cast<double*>(x.arena + x.plan->scratch_off[0]);
        k::GapBatch gb{};
        gb.n_seg = 1; gb.img_start[0] = 0; gb.img_start[1] = N; gb.seg[0] = gp;
        if (pool) {
          launch_pdl(k::gap_partial_f64, dim3(1, gp.slabs, N), dim3(256), 0, x.stream, gb);
          if (to_table) {          // slab partials -> sums (HW = 1: no division) in the table
            gb.seg[0].out = nullptr; gb.seg[0].out_f64 = sums; gb.seg[0].HW = 1;
            launch_pdl(k::gap_final_f64, dim3((N * gp.C + 7) / 8, 1), dim3(256), 0, x.stream, gb);
          }
        }
        k::GateParams q{};
        q.partial = to_table ? sums : gp.partial;
        q.w = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pw));
        q.b = reinterpret_cast<const __nv_bfloat16*>(x.resolve(pb));
        q.gate = reinterpret_cast<unsigned char*>(x.resolve(pg));
        q.z_out = want_z ? x.resolve(pz) : nullptr;
        q.z_bf16 = zb;
        q.C = gp.C; q.slabs = to_table ? 1 : gp.slabs; q.HW = gp.HW;
        if (fuse_part) {
          char* auxp = auxb + part_aux;
          q.ticket = reinterpret_cast<int*>(x.arena + 128) + ticket;
          q.part.gate = q.gate;
          q.part.n = N;
          q.part.idx_exec = reinterpret_cast<int*>(auxp);
          q.part.idx_skip = q.part.idx_exec + N;
          q.part.count_exec = reinterpret_cast<long long*>(x.arena + part_slot);
          q.part.count_skip = reinterpret_cast<long long*>(auxp + 2 * N * 4);
          q.zero_rows = zero_exec ? sums : nullptr;
        }
        // the sums table (or a few slabs per image): one CTA, a warp per image; many slabs: a CTA per image and a ticket
        if (q.slabs <= 4) launch_pdl(k::gate_logit_block_f64, dim3(1), dim3(1024), 0, x.stream, q, N);
        else launch_pdl(k::gate_logit_f64, dim3(N), dim3(256), 0, x.stream, q);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // ------------------------------------------------------------------------------ Switch / Combine
  Status build_switch(int gi, const Group& G) {
    if (p.n_req != 1) return fail(E_UNSUPPORTED_OP, "Switch/Combine graphs carry the batch inside the graph: bind one request");
    const View& vx = p.views[G.a][0];
    if (vx.dims.size() != 4 || !is_channels_last(vx)) return fail(E_UNSUPPORTED_OP, "Switch regroups channels-last samples");
    const int N = static_cast<int>(vx.dims[0]);
    const long long bytes = vx.dims[1] * vx.dims[2] * vx.dims[3] * dtype_size(g.tensors[G.a].dtype);
    if (bytes % 16) return fail(E_UNSUPPORTED_OP, "Switch: sample size must be a multiple of 16 bytes");
    RtCount rc = runtime_count(G.out, 0);
    if (!rc.rt || rc.a != 0 || rc.b != 1) return fail(E_INTERNAL, "Switch output has no run-time count");
    const bool fused = partition_fused.count(G.gate) != 0;   // the gate kernel has already partitioned the ids
    const size_t aux = fused ? switch_aux[G.gate] : aux_need;
    if (!fused) {
      switch_aux[G.gate] = aux;
      aux_need += (static_cast<size_t>(2 * N) * 4 + 16 + 255) & ~size_t(255);
      count_known_after(gi, G.out);
    }
    const bool indirect = c.storage[G.out].kind == Storage::INDIRECT_IN;
    if (fused && indirect) return OK;
    Ptr px = ptr_of(G.a, 0), pg = ptr_of(G.gate, 0), pe = ptr_of(G.out, 0);
    const bool has_skip = G.out2 >= 0 && !p.views[G.out2][0].dims.empty();
    Ptr ps = has_skip ? ptr_of(G.out2, 0) : Ptr();
    const size_t slot = rc.slot_off;
    add(gi, (has_skip ? 3 : 2) - (fused ? 1 : 0), [=](const RunCtx& x) {
      char* auxp = x.arena + x.plan->scratch_off[1] + aux;
      k::PartitionParams pp{};
      pp.gate = reinterpret_cast<const unsigned char*>(x.resolve(pg));
      pp.n = N;
      pp.idx_exec = reinterpret_cast<int*>(auxp);
      pp.idx_skip = pp.idx_exec + N;
      pp.count_exec = reinterpret_cast<long long*>(x.arena + slot);
      pp.count_skip = reinterpret_cast<long long*>(auxp + 2 * N * 4);
      if (!fused) launch_pdl(k::gate_partition, dim3(1), dim3(32), 0, x.stream, pp);
      if (indirect) return cudaGetLastError();   // the consumers read the Switch input through the id lists
      k::SampleCopyParams sc{};
      sc.src = reinterpret_cast<const uint4*>(x.resolve(px));
      sc.vec_per_sample = bytes / 16;
      sc.scatter = 0;
      const unsigned gx = static_cast<unsigned>(std::max<long long>(1, std::min<long long>(64, sc.vec_per_sample / 256)));
      sc.dst = reinterpret_cast<uint4*>(x.resolve(pe));
      sc.idx = pp.idx_exec;
      sc.count = pp.count_exec;
      launch_pdl(k::sample_copy, dim3(gx, N), dim3(256), 0, x.stream, sc);
      if (has_skip) {
        sc.dst = reinterpret_cast<uint4*>(x.resolve(ps));
        sc.idx = pp.idx_skip;
        sc.count = pp.count_skip;
        launch_pdl(k::sample_copy, dim3(gx, N), dim3(256), 0, x.stream, sc);
      }
      return cudaGetLastError();
    });
    return OK;
  }

  Status build_combine(int gi, const Group& G) {
    if (p.n_req != 1) return fail(E_UNSUPPORTED_OP, "Switch/Combine graphs carry the batch inside the graph: bind one request");
    auto it = switch_aux.find(G.gate);
    if (it == switch_aux.end()) return fail(E_INTERNAL, "Combine without a Switch on the same gate");
    const size_t aux = it->second;
    const View& vy = p.views[G.out][0];
    if (vy.dims.size() != 4 || !is_channels_last(vy)) return fail(E_UNSUPPORTED_OP, "Combine writes channels-last samples");
    const int N = static_cast<int>(vy.dims[0]);
    const long long bytes = vy.dims[1] * vy.dims[2] * vy.dims[3] * dtype_size(g.tensors[G.out].dtype);
    if (bytes % 16) return fail(E_UNSUPPORTED_OP, "Combine: sample size must be a multiple of 16 bytes");
    RtCount rc = runtime_count(G.a, 0);
    if (!rc.rt) return fail(E_INTERNAL, "Combine input has no run-time count");
    Ptr pe = ptr_of(G.a, 0), ps = ptr_of(G.res, 0), py = ptr_of(G.out, 0);
    const size_t slot = rc.slot_off;
    if (c.storage[G.a].kind == Storage::INDIRECT_OUT) {
      // the executed samples are already in place; the skipped ones move from the Switch input to the
      // same sample slots of the output
      if (c.storage[G.res].kind != Storage::INDIRECT_IN) return fail(E_INTERNAL, "Combine: indirect executed operand with a copied skipped operand");
      if (c.storage[G.out].kind == Storage::ALIAS) return OK;   // in place: every sample is already where it belongs
      add(gi, 1, [=](const RunCtx& x) {
        char* auxp = x.arena + x.plan->scratch_off[1] + aux;
        k::SampleCopyParams sc{};
        sc.dst = reinterpret_cast<uint4*>(x.resolve(py));
        sc.src = reinterpret_cast<const uint4*>(x.resolve(ps));
        sc.vec_per_sample = bytes / 16;
        sc.scatter = 2;
        sc.idx = reinterpret_cast<const int*>(auxp) + N;
        sc.count = reinterpret_cast<const long long*>(auxp + 2 * N * 4);
        const unsigned gx = static_cast<unsigned>(std::max<long long>(1, std::min<long long>(64, sc.vec_per_sample / 256)));
        launch_pdl(k::sample_copy, dim3(gx, N), dim3(256), 0, x.stream, sc);
        return cudaGetLastError();
      });
      return OK;
    }
    add(gi, 2, [=](const RunCtx& x) {
      char* auxp = x.arena + x.plan->scratch_off[1] + aux;
      k::SampleCopyParams sc{};
      sc.dst = reinterpret_cast<uint4*>(x.resolve(py));
      sc.vec_per_sample = bytes / 16;
      sc.scatter = 1;
      const unsigned gx = static_cast<unsigned>(std::max<long long>(1, std::min<long long>(64, sc.vec_per_sample / 256)));
      sc.src = reinterpret_cast<const uint4*>(x.resolve(pe));
      sc.idx = reinterpret_cast<const int*>(auxp);
      sc.count = reinterpret_cast<const long long*>(x.arena + slot);
      launch_pdl(k::sample_copy, dim3(gx, N), dim3(256), 0, x.stream, sc);
      sc.src = reinterpret_cast<const uint4*>(x.resolve(ps));
      sc.idx = reinterpret_cast<const int*>(auxp) + N;
      sc.count = reinterpret_cast<const long long*>(auxp + 2 * N * 4);
      launch_pdl(k::sample_copy, dim3(gx, N), dim3(256), 0, x.stream, sc);
      return cudaGetLastError();
    });
    return OK;
  }

  // ------------------------------------------------------------------------------ global average pool
  Status build_gap(int gi, const Group& G) {
    const Tensor& X = g.tensors[G.a];
    const Tensor& O = g.tensors[G.out];
    if (X.dtype != DType::BF16) return fail(E_UNSUPPORTED_OP, "global average pool is bf16 only");
    // the requests of a batch are pooled together, up to GAP_MAX_SEG per launch pair
    for (int r0 = 0; r0 < p.n_req; r0 += k::GAP_MAX_SEG) {
      k::GapBatch gb{};
      std::vector<Ptr> px, po;
      std::vector<size_t> poff;
      size_t part_bytes = 0;
      int max_slabs = 1, max_nc = 0;
      // about four CTAs per SM over the whole launch, shared among the images in proportion to their pixels: the
      // kernel streams at the HBM rate once it runs, and more, shorter CTAs only add to its fixed cost
      double total_px = 0.0;
      for (int r = r0; r < std::min(p.n_req, r0 + k::GAP_MAX_SEG); ++r) {
        const View& vx = p.views[G.a][r];
        if (numel(vx.dims)) total_px += static_cast<double>(vx.dims[0]) * static_cast<double>(vx.dims[2] * vx.dims[3]);
      }
      for (int r = r0; r < std::min(p.n_req, r0 + k::GAP_MAX_SEG); ++r) {
        const View& vx = p.views[G.a][r];
        if (!numel(vx.dims)) continue;
        if (!is_channels_last(vx)) return fail(E_UNSUPPORTED_OP, "global average pool reads channels-last storage");
        k::GapParams gp{};
        gp.C = static_cast<int>(vx.dims[1]);
        gp.HW = vx.dims[2] * vx.dims[3];
        const long long share = static_cast<long long>(std::ceil(592.0 * static_cast<double>(gp.HW) / total_px));
        gp.slabs = static_cast<int>(std::max<long long>(1, std::min<long long>(share, gp.HW / (vx.dims[0] >= 16 ? 16 : 128))));
        gp.out_bf16 = O.dtype == DType::BF16;
        const int N = static_cast<int>(vx.dims[0]);
        const int si = gb.n_seg++;
        gb.img_start[si + 1] = gb.img_start[si] + N;
        gb.seg[si] = gp;
        px.push_back(ptr_of(G.a, r)); po.push_back(ptr_of(G.out, r)); poff.push_back(part_bytes);
        part_bytes += static_cast<size_t>(N) * gp.slabs * gp.C * 8;
        max_slabs = std::max(max_slabs, gp.slabs);
        max_nc = std::max(max_nc, N * gp.C);
      }
      if (!gb.n_seg) continue;
      scratch_need = std::max(scratch_need, part_bytes);
      const int n_img = gb.img_start[gb.n_seg];
      add(gi, 2, [=](const RunCtx& x) mutable {
        for (int si = 0; si < gb.n_seg; ++si) {
          gb.seg[si].x = reinterpret_cast<const __nv_bfloat16*>(x.resolve(px[si]));
          gb.seg[si].partial = reinterpret_cast<double*>(x.arena + x.plan->scratch_off[0] + poff[si]);
          gb.seg[si].out = x.resolve(po[si]);
          gb.seg[si].out_f64 = nullptr;
        }
        launch_pdl(k::gap_partial_f64, dim3(1, max_slabs, n_img), dim3(256), 0, x.stream, gb);
        launch_pdl(k::gap_final_f64, dim3((max_nc + 7) / 8, gb.n_seg), dim3(256), 0, x.stream, gb);
        return cudaGetLastError();
      });
    }
    return OK;
  }

  // Algorithmic cost of a group for the bound shapes: every external input and output once,
  // constants once, nothing for intermediates inside the group; flops of its contraction.
  void cost(const Group& G) {
    double bytes = 0, flops = 0;
    auto tb = [&](int t) {
      const Tensor& T = g.tensors[t];
      double b = 0;
      const int nr = T.kind == TKind::CONST ? 1 : p.n_req;
      for (int r = 0; r < nr; ++r) b += static_cast<double>(numel(p.views[t][r].dims)) * dtype_size(T.dtype);
      return b;
    };
    for (int t : G.ext_in) if (c.storage[t].kind != Storage::FOLDED && !p.views[t][0].dims.empty()) bytes += tb(t);
    for (int t : G.ext_out) if (c.storage[t].kind != Storage::FOLDED && !p.views[t][0].dims.empty()) bytes += tb(t);
    // index-indirect regrouping moves less: the Switch only partitions the sample ids, the Combine
    // reads and writes the skipped samples (upper bound: all of them) and never touches the executed operand
    if (G.kind == GKind::SWITCH && c.storage[G.out].kind == Storage::INDIRECT_IN)
      bytes = tb(G.gate) + 2.0 * 4.0 * static_cast<double>(p.views[G.a][0].dims[0]);
    if (G.kind == GKind::COMBINE && c.storage[G.a].kind == Storage::INDIRECT_OUT)
      bytes = c.storage[G.out].kind == Storage::ALIAS ? 0.0 : tb(G.res) + tb(G.out) + tb(G.gate);
    if (G.kind == GKind::GEMM) {
      const Tensor& W = g.tensors[G.w];
      const double K = static_cast<double>(W.S.dims[0].e.const_value()), N = static_cast<double>(W.S.dims[1].e.const_value());
      for (int r = 0; r < p.n_req; ++r) flops += 2.0 * (numel(p.views[G.a][r].dims) / K) * N * K;
    } else if (G.kind == GKind::ATTENTION) {
      for (int r = 0; r < p.n_req; ++r) {
        const auto& d = p.views[G.q][r].dims;
        const double L = static_cast<double>(d[d.size() - 2]), dh = static_cast<double>(d.back());
        flops += 4.0 * L * L * dh * (numel(d) / (L * dh));
      }
    } else if (G.kind == GKind::CONV) {
      const auto& wd = g.tensors[G.w].S.dims;
      const double per_out = 2.0 * wd[1].e.const_value() * wd[2].e.const_value() * wd[3].e.const_value();
      const int conv_out = g.nodes[G.nodes[0]].outs[0];
      for (int r = 0; r < p.n_req; ++r)
        if (!p.b->dims[conv_out].empty()) flops += per_out * numel(p.b->dims[conv_out][r]);
    }
    p.group_flops.push_back(flops);
    p.group_bytes.push_back(bytes);
  }

  Status run() {
    p.launches.clear();
    p.group_flops.clear();
    p.group_bytes.clear();
    p.gpu_launches = 0;
    p.rt_syms_after.assign(c.groups.size(), {});
    // the fp32 row kernel and the elementwise chains have no bounded waits, tickets or device-side counts
    // a pooling group right after a layout change of the SAME tensor: neither reads what the other writes, and the
    // shared input stays live over both steps, so the arena plan (liveness by step) cannot hand the pooled output a
    // slot that the layout kernel still reads
    p.side_group.assign(c.groups.size(), 0);
    for (size_t gi = 1; gi < c.groups.size(); ++gi) {
      const Group &A = c.groups[gi - 1], &Bg = c.groups[gi];
      if (Bg.kind == GKind::GAP && A.kind == GKind::LAYOUT && Bg.a == A.a && Bg.a != A.out && A.a != Bg.out && !p.side_group[gi - 1])
        p.side_group[gi] = 1;
    }
    p.uses_header = false;
    for (const Group& G : c.groups)
      if (!((G.kind == GKind::GEMM && g.tensors[G.a].dtype == DType::F32) || G.kind == GKind::CHAIN || G.kind == GKind::BMM ||
            G.kind == GKind::SUMSQ || G.kind == GKind::TOPK || G.kind == GKind::GATHER || G.kind == GKind::FILL || G.kind == GKind::RESIZE)) p.uses_header = true;
    // SOD2_HOST_PROFILE: host time of building the launches, per group kind
    static const bool prof = getenv("SOD2_HOST_PROFILE") != nullptr;
    struct KindTimes {
      double us[32] = {0};
      int n[32] = {0};
      bool on;
      explicit KindTimes(bool o) : on(o) {}
      ~KindTimes() {
        if (!on) return;
        for (int k = 0; k < 32; ++k) if (n[k]) fprintf(stderr, "[sod2] launches: %-10s %3d groups %.1f us\n", gkind_name(static_cast<GKind>(k)), n[k], us[k]);
      }
    } kt(prof);
    for (size_t gi = 0; gi < c.groups.size(); ++gi) {
      const Group& G = c.groups[gi];
      Status s = OK;
      struct Tick {
        KindTimes& kt; int k; std::chrono::steady_clock::time_point q0;
        Tick(KindTimes& t, int kind) : kt(t), k(kind & 31) { if (kt.on) q0 = std::chrono::steady_clock::now(); }
        ~Tick() { if (kt.on) { kt.us[k] += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - q0).count(); ++kt.n[k]; } }
      } tick(kt, static_cast<int>(G.kind));
      if (gi < p.chain_of.size() && p.chain_of[gi] >= 0) {
        // the first member builds the launch for the whole chain
        if (p.chains[p.chain_of[gi]].groups.front() == static_cast<int>(gi)) s = build_gemm_chain(p.chain_of[gi]);
        if (s != OK) return s;
        cost(G);
        continue;
      }
      switch (G.kind) {
        case GKind::GEMM: s = build_gemm(static_cast<int>(gi), G); break;
        case GKind::ATTENTION: s = build_attention(static_cast<int>(gi), G); break;
        case GKind::LAYERNORM: s = build_layernorm(static_cast<int>(gi), G); break;
        case GKind::CHAIN: s = build_chain(static_cast<int>(gi), G); break;
        case GKind::TOPK_KEEP: s = build_topk(static_cast<int>(gi), G); break;
        case GKind::NONZERO: s = build_nonzero(static_cast<int>(gi), G); break;
        case GKind::LAYOUT: s = build_layout(static_cast<int>(gi), G); break;
        case GKind::CONV: s = build_conv(static_cast<int>(gi), G); break;
        case GKind::GAP: s = build_gap(static_cast<int>(gi), G); break;
        case GKind::GATE: s = build_gate(static_cast<int>(gi), G); break;
        case GKind::SWITCH: s = build_switch(static_cast<int>(gi), G); break;
        case GKind::COMBINE: s = build_combine(static_cast<int>(gi), G); break;
        case GKind::BMM: s = build_bmm(static_cast<int>(gi), G); break;
        case GKind::SUMSQ: s = build_sumsq(static_cast<int>(gi), G); break;
        case GKind::TOPK: s = build_topk_rows(static_cast<int>(gi), G); break;
        case GKind::GATHER: s = build_gather(static_cast<int>(gi), G); break;
        case GKind::FILL: s = build_fill(static_cast<int>(gi), G); break;
        case GKind::RESIZE: s = build_resize(static_cast<int>(gi), G); break;
        default: return fail(E_UNSUPPORTED_OP, std::string("no executor yet for group kind ") + gkind_name(G.kind));
      }
      if (s != OK) return s;
      cost(G);
    }
    if (p.front_reserve) {
      // staged plan: scratch and index lists at the fixed places behind the header that the first stage chose
      const size_t sc = (scratch_need + 255) & ~size_t(255), ax = (aux_need + 255) & ~size_t(255);
      if (sc > p.front_scratch || p.front_scratch + ax > p.front_reserve) return fail(E_INTERNAL, "stage needs more scratch than the bounded plan reserved");
      p.scratch_off.assign(2, p.header_end);
      p.scratch_off[1] = p.header_end + p.front_scratch;
      return OK;
    }
    // one scratch region shared by all groups (they run in stream order), after the tensors
    const size_t band = (c.flags & OPT_GUARD_BANDS) ? 256 : 0;
    p.scratch_off.assign(2, p.arena_bytes);
    p.arena_bytes += (scratch_need + 255) & ~size_t(255);
    if (band) { p.guard_bands.push_back({p.arena_bytes, -1}); p.arena_bytes += band; }
    p.scratch_off[1] = p.arena_bytes;     // index lists of Switch groups: live until their Combine
    p.arena_bytes += (aux_need + 255) & ~size_t(255);
    if (band) { p.guard_bands.push_back({p.arena_bytes, -2}); p.arena_bytes += band; }
    return OK;
  }
};

__global__ void transpose_bf16(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out, int K, int N) {
  // in [K, N] row-major -> out [N, K] row-major
  __shared__ __nv_bfloat16 tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int kk = k0 + i, n = n0 + threadIdx.x;
    if (kk < K && n < N) tile[i][threadIdx.x] = in[static_cast<long long>(kk) * N + n];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int n = n0 + i, kk = k0 + threadIdx.x;
    if (kk < K && n < N) out[static_cast<long long>(n) * K + kk] = tile[threadIdx.x][i];
  }
}

// Weights of a GEMM whose A operand is a folded LayerNorm: out[n, k] = bf16(gamma[k] * in[k, n]).
__global__ void transpose_scale_bf16(const __nv_bfloat16* __restrict__ in, const __nv_bfloat16* __restrict__ gamma,
                                     __nv_bfloat16* __restrict__ out, int K, int N) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int kk = k0 + i, n = n0 + threadIdx.x;
    if (kk < K && n < N) tile[i][threadIdx.x] = __float2bfloat16_rn(__bfloat162float(in[static_cast<long long>(kk) * N + n]) * __bfloat162float(gamma[kk]));
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int n = n0 + i, kk = k0 + threadIdx.x;
    if (kk < K && n < N) out[static_cast<long long>(n) * K + kk] = tile[threadIdx.x][i];
  }
}
// The two epilogue vectors of that GEMM, one warp per output column, fp64 sums in a fixed order:
//   c1[n] = sum_k Wp[n, k]  (of the scaled copy as rounded to bf16, so that it cancels what the MMA adds up)
//   c2[n] = sum_k beta[k] * W[k, n] + bias[n]
__global__ void ln_fold_vectors(const __nv_bfloat16* __restrict__ Wp, const __nv_bfloat16* __restrict__ W, const __nv_bfloat16* __restrict__ beta,
                                const __nv_bfloat16* __restrict__ bias, float* __restrict__ c1, float* __restrict__ c2, int K, int N) {
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  double a = 0.0, b = 0.0;
  for (int kk = lane; kk < K; kk += 32) {
    a += static_cast<double>(__bfloat162float(Wp[static_cast<long long>(n) * K + kk]));
    b += static_cast<double>(__bfloat162float(beta[kk])) * static_cast<double>(__bfloat162float(W[static_cast<long long>(kk) * N + n]));
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) { a += __shfl_xor_sync(0xffffffffu, a, o); b += __shfl_xor_sync(0xffffffffu, b, o); }
  if (lane == 0) {
    c1[n] = static_cast<float>(a);
    c2[n] = static_cast<float>(b + (bias ? static_cast<double>(__bfloat162float(bias[n])) : 0.0));
  }
}

}  // namespace

Status build_launches(Plan* p) {
  Builder b(*p);
  return b.run();
}

Status detect_chains(Plan* p) {
  Builder b(*p);
  return b.find_chains();
}

Status prepack_weights(Compiled* c, void* workspace, size_t bytes, void* stream) {
  if (c->packed_bytes == 0) { c->packed_ws = workspace; return OK; }
  if (!workspace || bytes < c->packed_bytes) { c->err = "prepack workspace too small"; return E_ARENA_TOO_SMALL; }
  if (reinterpret_cast<uintptr_t>(workspace) & 255) { c->err = "prepack workspace must be 256-byte aligned"; return E_MISALIGNED; }
  for (size_t i = 0; i < c->packed_consts.size(); ++i) {
    const Tensor& W = c->g.tensors[c->packed_consts[i]];
    if (!W.dev_ptr) { c->err = "constant " + W.name + " has no device data"; return E_INVALID_ARG; }
    if (W.S.rank == 4) {  // convolution weights [Cout, Cin, kh, kw] -> [Cout, (dy, dx, ci)]
      const int co = static_cast<int>(W.S.dims[0].e.const_value()), ci = static_cast<int>(W.S.dims[1].e.const_value());
      const int kh = static_cast<int>(W.S.dims[2].e.const_value()), kw = static_cast<int>(W.S.dims[3].e.const_value());
      bool stem = false;
      for (const Group& G2 : c->groups) if (G2.kind == GKind::CONV && G2.w == c->packed_consts[i] && is_fused_stem(*c, G2)) stem = true;
      if (stem) {     // fused RGB stem: (dy, ci, dx + 1) order, 24 units of 8
        k::reorder_stem_weights<<<48, 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __nv_bfloat16*>(W.dev_ptr), reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]));
        continue;
      }
      if (ci % 64) {  // thin-channel convolution (im2col path): keep the (ci, dy, dx) order, pad K with zeros
        const int K = ci * kh * kw, Kp = (K + 63) / 64 * 64;
        k::pad_rows_bf16<<<148 * 2, 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __nv_bfloat16*>(W.dev_ptr), reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]), co, K, Kp);
        continue;
      }
      if (kh == 3 && kw == 3) {  // 3x3: (dy, channel chunk, dx, ci) so that the dx taps of a chunk are adjacent
        k::reorder_conv3x3_rows<<<148 * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __nv_bfloat16*>(W.dev_ptr), reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]), co, ci);
        continue;
      }
      k::reorder_conv_weights<<<148 * 4, 256, 0, static_cast<cudaStream_t>(stream)>>>(
          static_cast<const __nv_bfloat16*>(W.dev_ptr), reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]), co, ci, kh, kw);
      continue;
    }
    const int K = static_cast<int>(W.S.dims[0].e.const_value()), N = static_cast<int>(W.S.dims[1].e.const_value());
    if (c->packed_ln[i].gamma >= 0) {   // folded LayerNorm: gamma-scaled copy + the two epilogue vectors
      const Compiled::PackedLn& e = c->packed_ln[i];
      const Tensor &Gm = c->g.tensors[e.gamma], &Bt = c->g.tensors[e.beta];
      const Tensor* Bi = e.bias >= 0 ? &c->g.tensors[e.bias] : nullptr;
      if (!Gm.dev_ptr || !Bt.dev_ptr || (Bi && !Bi->dev_ptr)) { c->err = "LayerNorm constants of " + W.name + " have no device data"; return E_INVALID_ARG; }
      __nv_bfloat16* Wp = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]);
      float* c1 = reinterpret_cast<float*>(static_cast<char*>(workspace) + c->packed_off[i] + ((static_cast<size_t>(N) * K * 2 + 255) & ~size_t(255)));
      transpose_scale_bf16<<<dim3((N + 31) / 32, (K + 31) / 32), dim3(32, 8), 0, static_cast<cudaStream_t>(stream)>>>(
          static_cast<const __nv_bfloat16*>(W.dev_ptr), static_cast<const __nv_bfloat16*>(Gm.dev_ptr), Wp, K, N);
      ln_fold_vectors<<<(N + 7) / 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(
          Wp, static_cast<const __nv_bfloat16*>(W.dev_ptr), static_cast<const __nv_bfloat16*>(Bt.dev_ptr),
          Bi ? static_cast<const __nv_bfloat16*>(Bi->dev_ptr) : nullptr, c1, c1 + N, K, N);
      continue;
    }
    transpose_bf16<<<dim3((N + 31) / 32, (K + 31) / 32), dim3(32, 8), 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __nv_bfloat16*>(W.dev_ptr), reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + c->packed_off[i]), K, N);
  }
  if (cudaGetLastError() != cudaSuccess) { c->err = "prepack launch failed"; return E_CUDA; }
  c->packed_ws = workspace;
  return OK;
}

Status run_plan_timed(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream,
                      float* group_ms, int n_groups, int reps) {
  if (reps < 1) { p->err = "reps must be at least 1"; return E_INVALID_ARG; }
  if (!group_ms || n_groups != static_cast<int>(p->c->groups.size())) { p->err = "group_ms must hold one float per group"; return E_INVALID_ARG; }
  if (arena_bytes < p->arena_bytes) { p->err = "arena too small"; return E_ARENA_TOO_SMALL; }
  if (reinterpret_cast<uintptr_t>(arena) & 255) { p->err = "arena must be 256-byte aligned"; return E_MISALIGNED; }
  RunCtx x{inputs, outputs, static_cast<char*>(arena), static_cast<char*>(p->c->packed_ws), static_cast<cudaStream_t>(stream), p};
  const size_t n = p->launches.size();
  std::vector<cudaEvent_t> ev(2 * n);
  for (auto& e : ev) if (cudaEventCreate(&e) != cudaSuccess) { p->err = "cudaEventCreate failed"; return E_CUDA; }
  if (p->uses_header) cudaMemsetAsync(arena, 0, p->header_clear_bytes, x.stream);
  Status st = OK;
  for (size_t i = 0; i < n && st == OK; ++i) {
    cudaEventRecord(ev[2 * i], x.stream);
    for (int r = 0; r < reps && st == OK; ++r)
      if (p->launches[i]->fn(x) != cudaSuccess) { p->err = "launch failed"; st = E_CUDA; }
    cudaEventRecord(ev[2 * i + 1], x.stream);
  }
  if (cudaStreamSynchronize(x.stream) != cudaSuccess) { p->err = "stream synchronize failed"; st = E_CUDA; }
  for (int g = 0; g < n_groups; ++g) group_ms[g] = 0.f;
  if (st == OK)
    for (size_t i = 0; i < n; ++i) {
      float ms = 0.f;
      cudaEventElapsedTime(&ms, ev[2 * i], ev[2 * i + 1]);
      ms /= static_cast<float>(reps);
      if (p->launches[i]->share.empty()) group_ms[p->launches[i]->group] += ms;
      else for (auto& sh : p->launches[i]->share) group_ms[sh.first] += ms * static_cast<float>(sh.second);   // a chain: by algorithmic flops
    }
  for (auto& e : ev) cudaEventDestroy(e);
  return st;
}

Plan::~Plan() {
  if (graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(graph_exec));
  if (capture_stream) cudaStreamDestroy(static_cast<cudaStream_t>(capture_stream));
  if (side_stream) cudaStreamDestroy(static_cast<cudaStream_t>(side_stream));
  if (ev_fork) cudaEventDestroy(static_cast<cudaEvent_t>(ev_fork));
  if (ev_join) cudaEventDestroy(static_cast<cudaEvent_t>(ev_join));
}

// The second stream and the two events of a plan with side groups (made outside any stream capture).
static bool ensure_side_stream(Plan* p) {
  bool any = false;
  for (char c : p->side_group) any = any || c;
  if (!any || p->side_stream) return true;
  cudaStream_t s;
  cudaEvent_t a, b;
  if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) return false;
  if (cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess || cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
    cudaStreamDestroy(s);
    return false;
  }
  p->side_stream = s; p->ev_fork = a; p->ev_join = b;
  return true;
}

Status run_plan_graph(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream,
                      int64_t* info) {
  const Graph& G = p->c->g;
  std::vector<const void*> key;
  key.reserve(G.inputs.size() + G.outputs.size() + 1);
  for (size_t i = 0; i < G.inputs.size(); ++i) key.push_back(inputs[i]);
  for (size_t i = 0; i < G.outputs.size(); ++i) key.push_back(outputs[i]);
  key.push_back(arena);
  auto t0 = std::chrono::steady_clock::now();
  int64_t captured = 0;
  if (!p->graph_exec || key != p->graph_key) {
    if (p->graph_exec) { cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(p->graph_exec)); p->graph_exec = nullptr; }
    if (!p->capture_stream) {
      cudaStream_t cs;
      if (cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) != cudaSuccess) { p->err = "cannot create the capture stream"; return E_CUDA; }
      p->capture_stream = cs;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(p->capture_stream);
    if (!ensure_side_stream(p)) { p->err = "cannot create the second stream"; return E_CUDA; }
    if (cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { p->err = "cannot begin the stream capture"; return E_CUDA; }
    Status s = run_plan(p, inputs, outputs, arena, arena_bytes, cs, nullptr);
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(cs, &graph);     // always ended, also after a failed launch
    if (s != OK) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return s; }
    if (e != cudaSuccess || !graph) { p->err = std::string("stream capture failed: ") + cudaGetErrorString(e); cudaGetLastError(); return E_CUDA; }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ei != cudaSuccess) { p->err = std::string("graph instantiation failed: ") + cudaGetErrorString(ei); cudaGetLastError(); return E_CUDA; }
    p->graph_exec = exec;
    p->graph_key = key;
    captured = 1;
  } else {
    if (arena_bytes < p->arena_bytes) { p->err = "arena too small"; return E_ARENA_TOO_SMALL; }
  }
  const cudaError_t el = cudaGraphLaunch(static_cast<cudaGraphExec_t>(p->graph_exec), static_cast<cudaStream_t>(stream));
  if (el != cudaSuccess) { p->err = std::string("graph launch failed: ") + cudaGetErrorString(el); return E_CUDA; }
  if (info) {
    info[0] = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    info[1] = p->gpu_launches;
    info[3] = captured;
  }
  return OK;
}

Status run_plan(Plan* p, const void* const* inputs, void* const* outputs, void* arena, size_t arena_bytes, void* stream, int64_t* info,
                int step_lo, int step_hi) {
  if (!arena && p->arena_bytes) { p->err = "arena is null"; return E_INVALID_ARG; }
  if (arena_bytes < p->arena_bytes) { p->err = "arena too small"; return E_ARENA_TOO_SMALL; }
  if (reinterpret_cast<uintptr_t>(arena) & 255) { p->err = "arena must be 256-byte aligned"; return E_MISALIGNED; }
  if (p->c->packed_bytes && !p->c->packed_ws) { p->err = "weights are not prepacked"; return E_INVALID_ARG; }
  auto t0 = std::chrono::steady_clock::now();
  if (!p->sm_count_known) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) p->sm_count = n;
    p->sm_count_known = true;
  }
  RunCtx x{inputs, outputs, static_cast<char*>(arena), static_cast<char*>(p->c->packed_ws), static_cast<cudaStream_t>(stream), p};
  if (p->uses_header && step_lo <= 0 && cudaMemsetAsync(arena, 0, p->header_clear_bytes, x.stream) != cudaSuccess) { p->err = "cannot clear the status word"; return E_CUDA; }
  if (!ensure_side_stream(p)) { p->err = "cannot create the second stream"; return E_CUDA; }
  const int n_groups = static_cast<int>(p->side_group.size());
  cudaStream_t side = static_cast<cudaStream_t>(p->side_stream);
  bool open_fork = false;
  int64_t enqueued = 0;
  for (size_t i = 0; i < p->launches.size(); ++i) {
    auto& L = p->launches[i];
    const int g = L->group;
    if (g < step_lo || g > step_hi) continue;
    enqueued += L->n_kernels;
    const bool first_of_group = i == 0 || p->launches[i - 1]->group != g;
    const bool last_of_group = i + 1 == p->launches.size() || p->launches[i + 1]->group != g;
    const bool on_side = side && g >= 0 && g < n_groups && p->side_group[g] && open_fork;
    if (side && first_of_group && !open_fork && g + 1 < n_groups && p->side_group[g + 1]) {
      // the next group runs beside this one: it may start as soon as everything before this group is done
      if (cudaEventRecord(static_cast<cudaEvent_t>(p->ev_fork), x.stream) != cudaSuccess ||
          cudaStreamWaitEvent(side, static_cast<cudaEvent_t>(p->ev_fork), 0) != cudaSuccess) { p->err = "fork failed"; return E_CUDA; }
      open_fork = true;
    }
    RunCtx xs = x;
    if (on_side) xs.stream = side;
    cudaError_t e = L->fn(xs);
    if (e == cudaSuccess && on_side && last_of_group) {
      if (cudaEventRecord(static_cast<cudaEvent_t>(p->ev_join), side) != cudaSuccess ||
          cudaStreamWaitEvent(x.stream, static_cast<cudaEvent_t>(p->ev_join), 0) != cudaSuccess) { p->err = "join failed"; return E_CUDA; }
      open_fork = false;
    }
    if (e != cudaSuccess) {
      if (open_fork) {   // never leave the second stream forked (a capture could not end)
        cudaEventRecord(static_cast<cudaEvent_t>(p->ev_join), side);
        cudaStreamWaitEvent(x.stream, static_cast<cudaEvent_t>(p->ev_join), 0);
      }
      p->err = std::string("launch failed in group ") + std::to_string(L->group) + ": " + cudaGetErrorString(e);
      return E_CUDA;
    }
  }
  if (open_fork) {       // a side group without launches: join all the same
    cudaEventRecord(static_cast<cudaEvent_t>(p->ev_join), side);
    cudaStreamWaitEvent(x.stream, static_cast<cudaEvent_t>(p->ev_join), 0);
  }
  if (info) {
    info[0] = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    info[1] = (step_lo <= 0 && step_hi >= (1 << 30)) ? p->gpu_launches : enqueued;
  }
  return OK;
}

// ---- guard bands (OPT_GUARD_BANDS): the arena behind the header is filled with 0xFF bytes (NaN in bf16 and fp32, so
// a read of memory nothing wrote shows in the results), and after a run every 256-byte band behind a tensor or scratch
// region must still hold them: a kernel that stored past the end of its tensor has damaged the band behind it.
namespace {
struct GuardList { const size_t* off; int n; };
__global__ void check_guard_bands(const char* arena, GuardList gl, unsigned long long* result) {
  // one warp per band: 64 words of 4 bytes; result[0] = damaged bands, result[1] = lowest damaged band index
  const int band = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (band >= gl.n) return;
  const unsigned* w = reinterpret_cast<const unsigned*>(arena + gl.off[band]);
  const bool bad = w[lane] != 0xFFFFFFFFu || w[lane + 32] != 0xFFFFFFFFu;
  if (__any_sync(0xffffffffu, bad) && lane == 0) {
    atomicAdd(result, 1ull);
    atomicMin(result + 1, static_cast<unsigned long long>(band));
  }
}
}  // namespace

Status poison_arena(const Plan* p, void* arena, size_t arena_bytes, void* stream) {
  if (arena_bytes < p->arena_bytes) return E_ARENA_TOO_SMALL;
  const size_t from = p->header_end ? p->header_end : 256;
  if (p->arena_bytes > from && cudaMemsetAsync(static_cast<char*>(arena) + from, 0xFF, p->arena_bytes - from, static_cast<cudaStream_t>(stream)) != cudaSuccess) return E_CUDA;
  return OK;
}

// n_bad: damaged bands; first_tensor: tensor id behind which the lowest damaged band lies (-1 scratch, -2 index lists,
// -3 none).  The library allocates no device memory: the band offsets reach the kernel through the arena header's
// unused bytes 32..127, twelve at a time, and the result comes back through bytes 16..31.  Synchronises the stream.
Status check_guards(const Plan* p, void* arena, void* stream, int* n_bad, int* first_tensor) {
  *n_bad = 0;
  *first_tensor = -3;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (p->guard_bands.empty()) return OK;
  // header bytes 16..31 take the result, bytes 32..127 twelve band offsets at a time
  char* hdr = static_cast<char*>(arena);
  unsigned long long init[2] = {0ull, ~0ull};
  if (cudaMemcpyAsync(hdr + 16, init, 16, cudaMemcpyHostToDevice, st) != cudaSuccess) return E_CUDA;
  const int per = 12;
  unsigned long long res[2] = {0, ~0ull};
  unsigned long long total_bad = 0;
  long long first_band = -1;
  for (size_t b0 = 0; b0 < p->guard_bands.size(); b0 += per) {
    size_t offs[per];
    const int n = static_cast<int>(std::min<size_t>(per, p->guard_bands.size() - b0));
    for (int i = 0; i < n; ++i) offs[i] = p->guard_bands[b0 + i].first;
    if (cudaMemcpyAsync(hdr + 16, init, 16, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(hdr + 32, offs, sizeof(size_t) * n, cudaMemcpyHostToDevice, st) != cudaSuccess) return E_CUDA;
    check_guard_bands<<<(n + 7) / 8, 256, 0, st>>>(hdr, GuardList{reinterpret_cast<const size_t*>(hdr + 32), n}, reinterpret_cast<unsigned long long*>(hdr + 16));
    if (cudaMemcpyAsync(res, hdr + 16, 16, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return E_CUDA;
    total_bad += res[0];
    if (res[0] && first_band < 0) first_band = static_cast<long long>(b0) + static_cast<long long>(res[1]);
  }
  *n_bad = static_cast<int>(total_bad);
  if (first_band >= 0) *first_tensor = p->guard_bands[static_cast<size_t>(first_band)].second;
  return OK;
}

// Exact handling of execution-determined extents (Section 3: the output shape of such an operator is known only
// after it ran; Section 4.3: the graph is partitioned there; Section 4.4.1: memory is planned once the sizes are
// known).  The groups run stage by stage; after a group that leaves a count on the device (the gate kernel that
// partitions the sample ids, a Switch that partitions them itself, a NonZero) the counts are
// read back (one copy + one stream synchronisation), the run-time symbols are bound to them, and the rest of the
// graph is planned again at the true sizes: tensors that already exist keep their places, the others are laid
// out around them.  info: [0] host ns, [1] kernels enqueued, [2] stages, [3] largest arena extent any stage laid out,
// [4] host ns spent binding and planning the stages.
Status run_exact(const Compiled* c, const Binding* b0, const Plan* bounded, const void* const* inputs, void* const* outputs, void* arena,
                 size_t arena_bytes, void* stream, int64_t* info, std::string* err) {
  auto t0 = std::chrono::steady_clock::now();
  const Graph& g = c->g;
  const int n_req = b0->n_req;
  const int n_groups = static_cast<int>(c->groups.size());
  // run-time symbols whose counts are on the device once a group has run (recorded by the bounded plan's builders)
  std::vector<std::vector<int>> syms_of(n_groups);
  for (int gi = 0; gi < n_groups && gi < static_cast<int>(bounded->rt_syms_after.size()); ++gi) syms_of[gi] = bounded->rt_syms_after[gi];
  // the places of scratch and index lists: sized by the bounded plan, fixed for every stage
  const size_t front_scratch = bounded->scratch_off[1] - bounded->scratch_off[0];
  const size_t front_total = front_scratch + (bounded->arena_bytes - bounded->scratch_off[1]);
  std::unique_ptr<Binding> bind(new Binding());
  std::unique_ptr<Plan> plan(new Plan());
  std::vector<std::vector<std::pair<int, int64_t>>> rt(n_req);
  int64_t plan_ns = 0, launches = 0, stages = 0;
  size_t peak_extent = 0;
  auto make_stage = [&](const Plan* prev, int first_step, int last_step) -> Status {
    auto tp = std::chrono::steady_clock::now();
    std::unique_ptr<Binding> nb(new Binding());
    Status s = rebind_runtime(*b0, rt, nb.get());
    if (s != OK) { *err = nb->err; return s; }
    std::unique_ptr<Plan> np(new Plan());
    np->front_reserve = front_total;
    np->front_scratch = front_scratch;
    np->place_from_step = first_step;
    np->place_until_step = last_step;
    if (prev)
      for (size_t t = 0; t < prev->roots.size(); ++t) {
        const RootBuf& R = prev->roots[t];
        if (R.where == RootBuf::ARENA && R.def_step >= 0 && R.def_step < first_step && R.last_step >= first_step) np->pinned.push_back({static_cast<int>(t), R.arena_off});
      }
    s = make_plan(c, nb.get(), np.get());
    if (s != OK) { *err = np->err; return s; }
    if (np->arena_bytes > arena_bytes) { *err = "arena too small for a stage planned around the tensors in place"; return E_ARENA_TOO_SMALL; }
    peak_extent = std::max(peak_extent, np->arena_bytes);
    np->sm_count = bounded->sm_count;
    np->sm_count_known = bounded->sm_count_known;
    bind = std::move(nb);
    plan = std::move(np);
    plan_ns += std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - tp).count();
    ++stages;
    return OK;
  };
  // stages: runs of groups up to and including one after which a count is known (a cut may fall inside a sub-graph
  // of the partition: the gate kernel already knows the count that sizes the Switch outputs)
  struct Stage { int first_step, last_step; std::vector<int> newly; };
  std::vector<Stage> plan_stages;
  {
    int lo = 0;
    for (int gi = 0; gi < n_groups; ++gi) {
      if (syms_of[gi].empty() && gi + 1 < n_groups) continue;
      plan_stages.push_back(Stage{lo, gi, syms_of[gi]});
      lo = gi + 1;
    }
  }
  const size_t n_atoms = g.cx.atoms.size();
  std::vector<long long> counts(n_atoms * static_cast<size_t>(n_req));
  for (size_t k = 0; k < plan_stages.size(); ++k) {
    const Stage& st = plan_stages[k];
    if (st.last_step < 0) continue;                       // no group in these sub-graphs
    Status s = make_stage(k ? plan.get() : nullptr, st.first_step, st.last_step);
    if (s != OK) return s;
    int64_t inf[8] = {0};
    s = run_plan(plan.get(), inputs, outputs, arena, arena_bytes, stream, inf, st.first_step, st.last_step);
    if (s != OK) { *err = plan->err; return s; }
    launches += inf[1];
    if (k + 1 >= plan_stages.size() || st.newly.empty()) continue;
    // read the counts and bind the symbols: the next stage is planned at the true sizes
    if (cudaMemcpyAsync(counts.data(), static_cast<const char*>(arena) + 256, counts.size() * 8, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)) != cudaSuccess ||
        cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { *err = "cannot read the run-time counts"; return E_CUDA; }
    for (int r = 0; r < n_req; ++r)
      for (int a : st.newly) rt[r].push_back({a, counts[static_cast<size_t>(a) * n_req + r]});
  }
  if (info) {
    info[0] = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    info[1] = launches;
    info[2] = stages;
    info[3] = static_cast<int64_t>(peak_extent);
    info[4] = plan_ns;
  }
  return OK;
}

}  // namespace sod2
