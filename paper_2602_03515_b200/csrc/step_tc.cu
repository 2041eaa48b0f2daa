// Launch plan of the tensor-core path of one step.  Layers are processed in chunks whose
// transient bf16 scratch (hi/lo split of M, first-side products, X) fits a byte budget; within a
// chunk every phase of Algorithm 1 is ONE grouped launch over all layers of the chunk:
//
//   momentum EMA (+ bf16 hi/lo of M)                       element-wise, per layer
//   factors   L <- b L + (1-b) G G^T , R <- b R + (1-b) G^T G          (Alg. 2)
//   [refresh of the layers that are due]                                (Alg. 1 lines 5-6)
//   fwd1      T_G = U^T G , T_M = U^T M            -> bf16 hi/lo        (Alg. 1 lines 8-9)
//   v2        V~ <- b2 V~ + (1-b2) (T_G V)^2        fused epilogue      (line 10)
//   scale     X = (T_M V) / sqrt(V~ + eps)          fused epilogue      (line 11)
//   back1     Y = U X
//   wwrite    W <- (1 - eta lambda) W - eta Y V^T   fused epilogue
//
// fp32 operands of the forward rotations (U, V, M, T) enter as a bf16 hi/lo pair and the
// products hi*hi + lo*hi + hi*lo are accumulated in tensor memory: a single bf16 rounding of
// the basis leaks the dominant gradient directions into every rotated coordinate at the 1e-3
// level, which for low-rank-plus-noise gradients is as large as the noise coordinates
// themselves.  The back rotation acts on X, whose entries are O(1) by construction, and uses
// single bf16 operands.
#include <algorithm>

#include "step_tc.h"

namespace br {

namespace {
constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
constexpr size_t kDefaultScratch = 4ull << 30;

struct LayerScratch {
  __nv_bfloat16 *Mh = nullptr, *Ml = nullptr, *TGh = nullptr, *TGl = nullptr, *TMh = nullptr, *TMl = nullptr,
                *X = nullptr;
};

size_t layer_scratch_bytes(const Layer& L) {
  const size_t one = align_up((size_t)L.d.m * L.d.n * 2);
  return (L.left && L.right) ? 7 * one : 3 * one;
}

struct Chunk {
  std::vector<int> ids;
  std::vector<LayerScratch> scr;
  TcPlan *factors = nullptr, *fwd1 = nullptr, *v2 = nullptr, *scale = nullptr, *back1 = nullptr, *wwrite = nullptr;
};

std::vector<std::vector<int>> make_chunks(const std::vector<Layer>& layers, const br_hparams& hp) {
  const size_t limit = hp.scratch_limit_bytes ? (size_t)hp.scratch_limit_bytes : kDefaultScratch;
  std::vector<std::vector<int>> out;
  size_t used = 0;
  for (int i = 0; i < (int)layers.size(); ++i) {
    if (!layers[i].use_tc) continue;
    const size_t b = layer_scratch_bytes(layers[i]);
    if (out.empty() || used + b > limit) { out.emplace_back(); used = 0; }
    out.back().push_back(i);
    used += b;
  }
  return out;
}

TcOperand op(const void* ptr, int64_t ld, int mn) {
  TcOperand o; o.ptr = ptr; o.ld = ld; o.mn_major = mn; return o;
}
TcOperand ring_op(const Layer& L, int mn) {
  TcOperand o; o.ptr = L.ring; o.ld = L.d.n; o.mn_major = mn;
  o.ring_slots = L.ring_slots; o.slot_stride_bytes = (int64_t)L.slot_stride;
  return o;
}

}  // namespace

struct TcStep {
  std::vector<Chunk> chunks;
  std::vector<TcPlan*> factor_plan;   // per layer, BR_ACCUM_ON_REFRESH only
  std::string err;
};

size_t tc_step_scratch_bytes(const std::vector<Layer>& layers, const br_hparams& hp) {
  size_t worst = 0;
  for (const auto& ids : make_chunks(layers, hp)) {
    size_t b = 0;
    for (int i : ids) b += layer_scratch_bytes(layers[i]);
    worst = std::max(worst, b);
  }
  return worst;
}

void tc_step_destroy(TcStep* t) {
  if (!t) return;
  for (Chunk& c : t->chunks)
    for (TcPlan* p : {c.factors, c.fwd1, c.v2, c.scale, c.back1, c.wwrite}) tc_plan_destroy(p);
  for (TcPlan* p : t->factor_plan) tc_plan_destroy(p);
  delete t;
}

static void factor_problems(const Layer& L, float beta, std::vector<TcProblem>* out) {
  const int64_t m = L.d.m, n = L.d.n;
  if (L.L) {      // L <- beta L + (1-beta) G G^T : both operands K-major views of G
    TcProblem q; q.Md = m; q.Nd = m; q.K = n; q.n_pairs = 1;
    q.A[0] = ring_op(L, 0); q.B[0] = ring_op(L, 0);
    q.epilogue = EPI_AXPBY_F32; q.alpha = 1.f - beta; q.beta = beta; q.D = L.L; q.ldd = m; q.tau_max = L.d.tau_max;
    out->push_back(q);
  }
  if (L.R) {      // R <- beta R + (1-beta) G^T G : both operands MN-major views of G
    TcProblem q; q.Md = n; q.Nd = n; q.K = m; q.n_pairs = 1;
    q.A[0] = ring_op(L, 1); q.B[0] = ring_op(L, 1);
    q.epilogue = EPI_AXPBY_F32; q.alpha = 1.f - beta; q.beta = beta; q.D = L.R; q.ldd = n; q.tau_max = L.d.tau_max;
    out->push_back(q);
  }
}

TcStep* tc_step_create(std::vector<Layer>& layers, const br_hparams& hp, char* scratch, size_t bytes,
                       int device, cudaStream_t s, const char** err) {
  static thread_local std::string last;
  if (err) *err = nullptr;
  auto chunk_ids = make_chunks(layers, hp);
  if (chunk_ids.empty()) return nullptr;
  auto fail = [&](TcStep* t, const std::string& m) -> TcStep* {
    last = m; if (err) *err = last.c_str(); tc_step_destroy(t); return nullptr;
  };
  if (!tc_supported(device)) { last = "tensor-core path needs an sm_100 device and cuTensorMapEncodeTiled"; if (err) *err = last.c_str(); return nullptr; }
  TcStep* t = new TcStep();
  t->factor_plan.assign(layers.size(), nullptr);
  const float beta_f = hp.beta_factor < 0.f ? hp.beta2 : hp.beta_factor;
  for (const auto& ids : chunk_ids) {
    Chunk c;
    c.ids = ids;
    size_t off = 0;
    auto take = [&](size_t numel) {
      __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(scratch + off);
      off += align_up(numel * 2);
      return p;
    };
    std::vector<TcProblem> factors, fwd1, v2, scale, back1, wwrite;
    for (int i : ids) {
      const Layer& L = layers[i];
      const int64_t m = L.d.m, n = L.d.n, mn = m * n;
      LayerScratch S;
      S.Mh = take(mn); S.Ml = take(mn); S.X = take(mn);
      if (L.left && L.right) { S.TGh = take(mn); S.TGl = take(mn); S.TMh = take(mn); S.TMl = take(mn); }
      c.scr.push_back(S);
      const int tm = L.d.tau_max;
      if (L.d.src == BR_SRC_SECOND && hp.accum == BR_ACCUM_EVERY_STEP) factor_problems(L, beta_f, &factors);
      if (L.left && L.right) {
        {  // T_G = U^T G : (Uh, G) + (Ul, G); U and G both enter MN-major (contraction over rows)
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 2; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 1); q.B[0] = ring_op(L, 1);
          q.A[1] = op(L.Ul, m, 1); q.B[1] = ring_op(L, 1);
          q.epilogue = EPI_SPLIT_BF16; q.Dh = S.TGh; q.Dl = S.TGl; q.ldh = n;
          fwd1.push_back(q);
        }
        {  // T_M = U^T M : (Uh, Mh) + (Ul, Mh) + (Uh, Ml)
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 3; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 1); q.B[0] = op(S.Mh, n, 1);
          q.A[1] = op(L.Ul, m, 1); q.B[1] = op(S.Mh, n, 1);
          q.A[2] = op(L.Uh, m, 1); q.B[2] = op(S.Ml, n, 1);
          q.epilogue = EPI_SPLIT_BF16; q.Dh = S.TMh; q.Dl = S.TMl; q.ldh = n;
          fwd1.push_back(q);
        }
        for (int which = 0; which < 2; ++which) {   // (T V): T K-major, V MN-major
          TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 3; q.tau_max = tm;
          const __nv_bfloat16* Th = which ? S.TMh : S.TGh;
          const __nv_bfloat16* Tl = which ? S.TMl : S.TGl;
          q.A[0] = op(Th, n, 0); q.B[0] = op(L.Vh, n, 1);
          q.A[1] = op(Tl, n, 0); q.B[1] = op(L.Vh, n, 1);
          q.A[2] = op(Th, n, 0); q.B[2] = op(L.Vl, n, 1);
          q.D = L.V2; q.ldd = n;
          if (!which) { q.epilogue = EPI_SECOND_MOMENT; q.alpha = 1.f - hp.beta2; q.beta = hp.beta2; v2.push_back(q); }
          else { q.epilogue = EPI_SCALE_BF16; q.eps = hp.eps; q.Dh = S.X; q.ldh = n; scale.push_back(q); }
        }
        {  // Y = U X : U K-major, X MN-major; Y reuses the T_G buffer
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 1; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 0); q.B[0] = op(S.X, n, 1);
          q.epilogue = EPI_SPLIT_BF16; q.Dh = S.TGh; q.Dl = nullptr; q.ldh = n;
          back1.push_back(q);
        }
        {  // W <- decay W - eta Y V^T : both K-major
          TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 1; q.tau_max = tm;
          q.A[0] = op(S.TGh, n, 0); q.B[0] = op(L.Vh, n, 0);
          q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
          wwrite.push_back(q);
        }
      } else if (L.left) {
        {  // V~ from U^T G
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 2; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 1); q.B[0] = ring_op(L, 1);
          q.A[1] = op(L.Ul, m, 1); q.B[1] = ring_op(L, 1);
          q.epilogue = EPI_SECOND_MOMENT; q.alpha = 1.f - hp.beta2; q.beta = hp.beta2; q.D = L.V2; q.ldd = n;
          v2.push_back(q);
        }
        {  // X from U^T M
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 3; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 1); q.B[0] = op(S.Mh, n, 1);
          q.A[1] = op(L.Ul, m, 1); q.B[1] = op(S.Mh, n, 1);
          q.A[2] = op(L.Uh, m, 1); q.B[2] = op(S.Ml, n, 1);
          q.epilogue = EPI_SCALE_BF16; q.eps = hp.eps; q.D = L.V2; q.ldd = n; q.Dh = S.X; q.ldh = n;
          scale.push_back(q);
        }
        {  // W <- decay W - eta U X
          TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 1; q.tau_max = tm;
          q.A[0] = op(L.Uh, m, 0); q.B[0] = op(S.X, n, 1);
          q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
          wwrite.push_back(q);
        }
      } else {
        {  // V~ from G V
          TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 2; q.tau_max = tm;
          q.A[0] = ring_op(L, 0); q.B[0] = op(L.Vh, n, 1);
          q.A[1] = ring_op(L, 0); q.B[1] = op(L.Vl, n, 1);
          q.epilogue = EPI_SECOND_MOMENT; q.alpha = 1.f - hp.beta2; q.beta = hp.beta2; q.D = L.V2; q.ldd = n;
          v2.push_back(q);
        }
        {  // X from M V
          TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 3; q.tau_max = tm;
          q.A[0] = op(S.Mh, n, 0); q.B[0] = op(L.Vh, n, 1);
          q.A[1] = op(S.Ml, n, 0); q.B[1] = op(L.Vh, n, 1);
          q.A[2] = op(S.Mh, n, 0); q.B[2] = op(L.Vl, n, 1);
          q.epilogue = EPI_SCALE_BF16; q.eps = hp.eps; q.D = L.V2; q.ldd = n; q.Dh = S.X; q.ldh = n;
          scale.push_back(q);
        }
        {  // W <- decay W - eta X V^T
          TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 1; q.tau_max = tm;
          q.A[0] = op(S.X, n, 0); q.B[0] = op(L.Vh, n, 0);
          q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
          wwrite.push_back(q);
        }
      }
    }
    if (off > bytes) return fail(t, "tensor-core scratch is smaller than the plan needs");
    const char* perr = nullptr;
    auto build = [&](std::vector<TcProblem>& v, TcPlan** dst) -> bool {
      if (v.empty()) return true;
      *dst = tc_plan_create(v.data(), (int)v.size(), device, s, &perr);
      return *dst != nullptr;
    };
    t->chunks.push_back(c);
    Chunk& cc = t->chunks.back();
    if (!build(factors, &cc.factors) || !build(fwd1, &cc.fwd1) || !build(v2, &cc.v2) || !build(scale, &cc.scale) ||
        !build(back1, &cc.back1) || !build(wwrite, &cc.wwrite))
      return fail(t, perr ? perr : "plan creation failed");
  }
  if (hp.accum == BR_ACCUM_ON_REFRESH) {
    for (size_t i = 0; i < layers.size(); ++i) {
      const Layer& L = layers[i];
      if (!L.use_tc || L.d.src != BR_SRC_SECOND) continue;
      std::vector<TcProblem> f;
      factor_problems(L, beta_f, &f);
      const char* perr = nullptr;
      if (!f.empty() && !(t->factor_plan[i] = tc_plan_create(f.data(), (int)f.size(), device, s, &perr)))
        return fail(t, perr ? perr : "plan creation failed");
    }
  }
  return t;
}

int tc_step_run(TcStep* t, std::vector<Layer>& layers, const std::vector<const void*>& G, long long calls,
                int tau, const br_hparams& hp, int* d_status, cudaStream_t s, LaunchStats* stats,
                const TcStepCallbacks& cb, const char** err) {
  static thread_local std::string last;
  auto cuda_fail = [&](const char* what, cudaError_t e) {
    last = std::string(what) + ": " + cudaGetErrorString(e);
    if (err) *err = last.c_str();
    return (int)BR_ERR_CUDA;
  };
  const float dyn_alpha = -hp.lr, dyn_beta = 1.0f - hp.lr * hp.weight_decay;
  for (Chunk& c : t->chunks) {
    bool any = false;
    for (size_t j = 0; j < c.ids.size(); ++j) {
      Layer& L = layers[c.ids[j]];
      const void* g = G[c.ids[j]];
      if (!g) continue;
      any = true;
      // Alg. 1 line 4, with the bf16 hi/lo pair of the new M for the rotation
      const int span = stats->prof.begin(PROF_EMA, s);
      cudaError_t e = ema_momentum(L.M, g, 1, L.d.m * L.d.n, hp.beta1, nullptr, c.scr[j].Mh, c.scr[j].Ml, s);
      stats->prof.end(span, s, 14.0 * (double)L.d.m * (double)L.d.n);
      if (e != cudaSuccess) return cuda_fail("ema_momentum", e);
      stats->launches += 1;
    }
    if (!any) continue;
    auto launch = [&](TcPlan* p, const char* what) -> int {
      if (!p) return 0;
      const int span = stats->prof.begin(PROF_TC, s);
      cudaError_t e = tc_plan_launch(p, calls, tau, dyn_alpha, dyn_beta, d_status, s);
      stats->prof.end(span, s, tc_plan_flops(p));
      if (e != cudaSuccess) return cuda_fail(what, e);
      stats->launches += 1;
      stats->gemm_flops += tc_plan_flops(p);
      return 0;
    };
    int rc;
    if ((rc = launch(c.factors, "factor launch"))) return rc;
    std::vector<int> due;
    for (int i : c.ids) {
      Layer& L = layers[i];
      if (!G[i] || L.t % L.freq != 0) continue;
      if (t->factor_plan[i] && (rc = launch(t->factor_plan[i], "factor launch"))) return rc;
      due.push_back(i);
    }
    if (!due.empty()) {
      rc = cb.refresh(cb.ctx, due.data(), (int)due.size());
      if (rc != 0) { if (err) *err = nullptr; return rc; }
    }
    if ((rc = launch(c.fwd1, "first-side rotation launch"))) return rc;
    if ((rc = launch(c.v2, "second-moment launch"))) return rc;
    if ((rc = launch(c.scale, "scaling launch"))) return rc;
    if ((rc = launch(c.back1, "back-rotation launch"))) return rc;
    if ((rc = launch(c.wwrite, "weight-write launch"))) return rc;
  }
  return 0;
}

}  // namespace br

// ---------------------------------------------------------------------------------------------
// Stand-alone contraction entry point
// ---------------------------------------------------------------------------------------------
extern "C" br_status br_gemm_bf16(void* cuda_stream, int64_t Md, int64_t Nd, int64_t K, int n_pairs,
                                  const void* const* A, const void* const* B, int a_mn, int b_mn,
                                  int64_t lda, int64_t ldb, float* D, int64_t ldd, float alpha, float beta) {
  using namespace br;
  if (!A || !B || !D || n_pairs < 1 || n_pairs > 3) return BR_ERR_INVALID;
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || !tc_supported(device)) return BR_ERR_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  TcProblem q;
  q.Md = Md; q.Nd = Nd; q.K = K; q.n_pairs = n_pairs;
  for (int p = 0; p < n_pairs; ++p) {
    q.A[p].ptr = A[p]; q.A[p].ld = lda; q.A[p].mn_major = a_mn ? 1 : 0;
    q.B[p].ptr = B[p]; q.B[p].ld = ldb; q.B[p].mn_major = b_mn ? 1 : 0;
  }
  q.epilogue = EPI_AXPBY_F32; q.alpha = alpha; q.beta = beta; q.D = D; q.ldd = ldd;
  const char* err = nullptr;
  TcPlan* plan = tc_plan_create(&q, 1, device, s, &err);
  if (!plan) return BR_ERR_SHAPE;
  int* d_status = nullptr;
  br_status rc = BR_OK;
  if (cudaMalloc(&d_status, sizeof(int)) != cudaSuccess) { tc_plan_destroy(plan); return BR_ERR_OOM; }
  cudaMemsetAsync(d_status, 0, sizeof(int), s);
  if (tc_plan_launch(plan, 1, 0, alpha, beta, d_status, s) != cudaSuccess) rc = BR_ERR_CUDA;
  int word = 0;
  if (cudaStreamSynchronize(s) != cudaSuccess) rc = BR_ERR_CUDA;
  else if (cudaMemcpy(&word, d_status, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess && word < 0) rc = (br_status)word;
  cudaFree(d_status);
  tc_plan_destroy(plan);
  return rc;
}
