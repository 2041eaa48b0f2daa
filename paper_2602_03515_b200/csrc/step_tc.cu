// Launch plan of the tensor-core path of one step.
//
// Between two refreshes the bases U, V are constant, so the rotated momentum obeys
//   M~_t = U^T M_t V = beta1 M~_{t-1} + (1 - beta1) U^T G_t V
// exactly (Alg. 1 (momentum update) is linear).  The tensor-core path therefore keeps M~ as its state instead
// of M: the momentum is never rotated, which removes one of the four two-sided products of Alg. 1,
// and its EMA joins the second-moment update and the Adam scaling in one fused epilogue.  Only a
// refresh needs M itself: the due layers are re-expressed, M = U M~ V^T with the old basis before
// the refresh (Alg. 2 with S = 1st reads M) and M~ = U^T M V with the new basis after it.
//
// Layers are processed in chunks whose transient bf16 scratch fits a byte budget; within a chunk
// every phase is ONE grouped launch over all layers of the chunk:
//
//   factors   L <- b L + (1-b) G G^T , R <- b R + (1-b) G^T G            (Alg. 2)
//   [refresh of the layers that are due, bracketed by the re-expression]  (Alg. 1 (periodic refresh))
//   fwd1      T = U^T G  (or T = G V when n > m: the larger side first) -> bf16 hi/lo   (Alg. 1 (rotation of G), first side)
//   adam      G~ = T V, fused epilogue: M~ <- b1 M~ + (1-b1) G~ ; V~ <- b2 V~ + (1-b2) G~^2 ;
//             X = M~ / sqrt(V~ + eps)                                      (momentum, rotation, second moment, weight update)
//   back1     Y = U X
//   wwrite    W <- (1 - eta lambda) W - eta Y V^T     fused epilogue      (weight update)
//
// fp32 operands of the forward rotations (U, V, T, and M / M~ in the re-expression) enter as a
// bf16 hi/lo pair and the products hi*hi + lo*hi + hi*lo are accumulated in tensor memory: a single
// bf16 rounding of the basis leaks the dominant gradient directions into every rotated coordinate
// at the 1e-3 level, which for low-rank-plus-noise gradients is as large as the noise coordinates
// themselves.  The back rotation acts on X, whose entries are O(1) by construction, and uses
// single bf16 operands.
#include <algorithm>

#include "step_tc.h"

namespace br {

namespace {
constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
// Transient scratch of one chunk of layers.  Smaller chunks mean more launches but let more of what one
// phase writes (first-side products, X, Y) still be in L2 when the next phase reads it: on the ~3B layer
// set a step takes 158 ms with 8 GiB (3 chunks), 150 with 4, 147 with 2, 148 with 1, 150.5 with 0.5.
constexpr size_t kDefaultScratch = 2ull << 30;
// Factor products are accumulated in chunks of a few 64-deep k-blocks (see gemm_tc.cu, folded form): at
// least ten chunks per contraction where it is long enough, at most four k-blocks per chunk (the epilogue
// warps keep up with the tensor core from four k-blocks on; with two they are the limit: a step of the
// ~3B layer set takes 4 % longer with four than without the folding, 12 % longer with two).
inline int fold_kb(int64_t K) { return (int)std::max<int64_t>(1, std::min<int64_t>(4, (K + 63) / 64 / 10)); }

struct LayerScratch {
  __nv_bfloat16* B[4] = {nullptr, nullptr, nullptr, nullptr};
};

size_t layer_scratch_bytes(const Layer& L) {
  const size_t one = align_up((size_t)L.d.m * L.d.n * 2);
  return (L.left && L.right) ? 4 * one : 2 * one;
}

// The four phases of a re-expression: M = U M~ V^T (back) and M~ = U^T M V (fwd), each with a
// first-side product into a bf16 hi/lo pair and a second-side product into the fp32 buffer.
struct RxPlans {
  TcPlan *back1 = nullptr, *back2 = nullptr, *fwd1 = nullptr, *fwd2 = nullptr;
};

struct Chunk {
  std::vector<int> ids;
  std::vector<LayerScratch> scr;
  TcPlan *factors = nullptr, *fwd1 = nullptr, *adam = nullptr, *back1 = nullptr, *wwrite = nullptr;
  RxPlans rx;                       // all layers of the chunk
  std::vector<RxPlans> rx_layer;    // one layer at a time
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

// hi*hi + lo*hi + hi*lo for (A, B) given as hi/lo pairs
void three_pairs(TcProblem& q, const void* Ah, const void* Al, int64_t lda, int a_mn, const void* Bh,
                 const void* Bl, int64_t ldb, int b_mn) {
  q.n_pairs = 3;
  q.A[0] = op(Ah, lda, a_mn); q.B[0] = op(Bh, ldb, b_mn);
  q.A[1] = op(Al, lda, a_mn); q.B[1] = op(Bh, ldb, b_mn);
  q.A[2] = op(Ah, lda, a_mn); q.B[2] = op(Bl, ldb, b_mn);
}

void factor_problems(const Layer& L, float beta, std::vector<TcProblem>* out) {
  const int64_t m = L.d.m, n = L.d.n;
  if (L.L) {      // L <- beta L + (1-beta) G G^T : both operands K-major views of G
    TcProblem q; q.Md = m; q.Nd = m; q.K = n; q.n_pairs = 1;
    q.A[0] = ring_op(L, 0); q.B[0] = ring_op(L, 0);
    q.epilogue = EPI_AXPBY_F32; q.alpha = 1.f - beta; q.beta = beta; q.D = L.L; q.ldd = m; q.tau_max = L.d.tau_max;
    q.symmetric = 1; q.fold_kb = fold_kb(n);
    out->push_back(q);
  }
  if (L.R) {      // R <- beta R + (1-beta) G^T G : both operands MN-major views of G
    TcProblem q; q.Md = n; q.Nd = n; q.K = m; q.n_pairs = 1;
    q.A[0] = ring_op(L, 1); q.B[0] = ring_op(L, 1);
    q.epilogue = EPI_AXPBY_F32; q.alpha = 1.f - beta; q.beta = beta; q.D = L.R; q.ldd = n; q.tau_max = L.d.tau_max;
    q.symmetric = 1; q.fold_kb = fold_kb(m);
    out->push_back(q);
  }
}

struct StepProblems {
  std::vector<TcProblem> factors, fwd1, adam, back1, wwrite;
};
struct RxProblems {
  std::vector<TcProblem> back1, back2, fwd1, fwd2;
};

void rotated_adam_epilogue(TcProblem& q, const Layer& L, const br_hparams& hp, __nv_bfloat16* X) {
  q.epilogue = EPI_ROTATED_ADAM;
  q.alpha = 1.f - hp.beta2; q.beta = hp.beta2; q.beta1 = hp.beta1; q.eps = hp.eps;
  q.D = L.V2; q.D2 = L.M; q.ldd = L.d.n; q.Dh = X; q.ldh = L.d.n;
}

void step_problems(const Layer& L, const LayerScratch& S, const br_hparams& hp, StepProblems* P) {
  const int64_t m = L.d.m, n = L.d.n;
  const int tm = L.d.tau_max;
  if (L.left && L.right) {
    // The first side costs two products (the gradient is bf16 already), the second three (both
    // operands are hi/lo pairs): mn (4 d1 + 6 d2) flop for side orders d1, d2.  The larger side goes first.
    if (n > m) {
      {  // T = G V : G K-major, V MN-major
        TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 2; q.tau_max = tm;
        q.A[0] = ring_op(L, 0); q.B[0] = op(L.Vh, n, 1);
        q.A[1] = ring_op(L, 0); q.B[1] = op(L.Vl, n, 1);
        q.epilogue = EPI_SPLIT_BF16; q.Dh = S.B[0]; q.Dl = S.B[1]; q.ldh = n;
        P->fwd1.push_back(q);
      }
      {  // G~ = U^T T : both MN-major (contraction over rows)
        TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.tau_max = tm;
        three_pairs(q, L.Uh, L.Ul, m, 1, S.B[0], S.B[1], n, 1);
        rotated_adam_epilogue(q, L, hp, S.B[2]);
        P->adam.push_back(q);
      }
    } else {
      {  // T = U^T G : (Uh, G) + (Ul, G); U and G both enter MN-major (contraction over rows)
        TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 2; q.tau_max = tm;
        q.A[0] = op(L.Uh, m, 1); q.B[0] = ring_op(L, 1);
        q.A[1] = op(L.Ul, m, 1); q.B[1] = ring_op(L, 1);
        q.epilogue = EPI_SPLIT_BF16; q.Dh = S.B[0]; q.Dl = S.B[1]; q.ldh = n;
        P->fwd1.push_back(q);
      }
      {  // G~ = T V : T K-major, V MN-major
        TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.tau_max = tm;
        three_pairs(q, S.B[0], S.B[1], n, 0, L.Vh, L.Vl, n, 1);
        rotated_adam_epilogue(q, L, hp, S.B[2]);
        P->adam.push_back(q);
      }
    }
    {  // Y = U X : U K-major, X MN-major
      TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 1; q.tau_max = tm;
      q.A[0] = op(L.Uh, m, 0); q.B[0] = op(S.B[2], n, 1);
      q.epilogue = EPI_SPLIT_BF16; q.Dh = S.B[0]; q.Dl = nullptr; q.ldh = n;
      P->back1.push_back(q);
    }
    {  // W <- decay W - eta Y V^T : both K-major
      TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 1; q.tau_max = tm;
      q.A[0] = op(S.B[0], n, 0); q.B[0] = op(L.Vh, n, 0);
      q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
      P->wwrite.push_back(q);
    }
  } else if (L.left) {
    {  // G~ = U^T G
      TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 2; q.tau_max = tm;
      q.A[0] = op(L.Uh, m, 1); q.B[0] = ring_op(L, 1);
      q.A[1] = op(L.Ul, m, 1); q.B[1] = ring_op(L, 1);
      rotated_adam_epilogue(q, L, hp, S.B[0]);
      P->adam.push_back(q);
    }
    {  // W <- decay W - eta U X
      TcProblem q; q.Md = m; q.Nd = n; q.K = m; q.n_pairs = 1; q.tau_max = tm;
      q.A[0] = op(L.Uh, m, 0); q.B[0] = op(S.B[0], n, 1);
      q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
      P->wwrite.push_back(q);
    }
  } else {
    {  // G~ = G V
      TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 2; q.tau_max = tm;
      q.A[0] = ring_op(L, 0); q.B[0] = op(L.Vh, n, 1);
      q.A[1] = ring_op(L, 0); q.B[1] = op(L.Vl, n, 1);
      rotated_adam_epilogue(q, L, hp, S.B[0]);
      P->adam.push_back(q);
    }
    {  // W <- decay W - eta X V^T
      TcProblem q; q.Md = m; q.Nd = n; q.K = n; q.n_pairs = 1; q.tau_max = tm;
      q.A[0] = op(S.B[0], n, 0); q.B[0] = op(L.Vh, n, 0);
      q.epilogue = EPI_AXPBY_F32; q.dyn_scalars = 1; q.D = L.d.weight; q.ldd = n;
      P->wwrite.push_back(q);
    }
  }
}

// Re-expression problems.  The fp32 buffer L.M is split into the bf16 pair (B0, B1) by the caller
// before either direction; the first-side product of a bilateral layer goes to (B2, B3).
void rx_problems(const Layer& L, const LayerScratch& S, RxProblems* P) {
  const int64_t m = L.d.m, n = L.d.n;
  auto store_f32 = [&](TcProblem& q) {
    q.epilogue = EPI_AXPBY_F32; q.alpha = 1.f; q.beta = 0.f; q.D = L.M; q.ldd = n;
  };
  auto store_pair = [&](TcProblem& q) {
    q.epilogue = EPI_SPLIT_BF16; q.Dh = S.B[2]; q.Dl = S.B[3]; q.ldh = n;
  };
  if (L.left && L.right) {
    { TcProblem q; q.Md = m; q.Nd = n; q.K = m;      // Y = U M~ : U K-major, M~ MN-major
      three_pairs(q, L.Uh, L.Ul, m, 0, S.B[0], S.B[1], n, 1); store_pair(q); P->back1.push_back(q); }
    { TcProblem q; q.Md = m; q.Nd = n; q.K = n;      // M = Y V^T : both K-major
      three_pairs(q, S.B[2], S.B[3], n, 0, L.Vh, L.Vl, n, 0); store_f32(q); P->back2.push_back(q); }
    { TcProblem q; q.Md = m; q.Nd = n; q.K = m;      // T = U^T M : both MN-major
      three_pairs(q, L.Uh, L.Ul, m, 1, S.B[0], S.B[1], n, 1); store_pair(q); P->fwd1.push_back(q); }
    { TcProblem q; q.Md = m; q.Nd = n; q.K = n;      // M~ = T V : T K-major, V MN-major
      three_pairs(q, S.B[2], S.B[3], n, 0, L.Vh, L.Vl, n, 1); store_f32(q); P->fwd2.push_back(q); }
  } else if (L.left) {
    { TcProblem q; q.Md = m; q.Nd = n; q.K = m;      // M = U M~
      three_pairs(q, L.Uh, L.Ul, m, 0, S.B[0], S.B[1], n, 1); store_f32(q); P->back2.push_back(q); }
    { TcProblem q; q.Md = m; q.Nd = n; q.K = m;      // M~ = U^T M
      three_pairs(q, L.Uh, L.Ul, m, 1, S.B[0], S.B[1], n, 1); store_f32(q); P->fwd2.push_back(q); }
  } else {
    { TcProblem q; q.Md = m; q.Nd = n; q.K = n;      // M = M~ V^T
      three_pairs(q, S.B[0], S.B[1], n, 0, L.Vh, L.Vl, n, 0); store_f32(q); P->back2.push_back(q); }
    { TcProblem q; q.Md = m; q.Nd = n; q.K = n;      // M~ = M V
      three_pairs(q, S.B[0], S.B[1], n, 0, L.Vh, L.Vl, n, 1); store_f32(q); P->fwd2.push_back(q); }
  }
}

void destroy(RxPlans& r) {
  for (TcPlan* p : {r.back1, r.back2, r.fwd1, r.fwd2}) tc_plan_destroy(p);
  r = RxPlans{};
}

}  // namespace

struct TcStep {
  std::vector<Chunk> chunks;
  std::vector<TcPlan*> factor_plan;   // per layer, BR_ACCUM_ON_REFRESH only
  std::vector<int> chunk_of, slot_of; // per layer: its chunk and its position in the chunk
  const float* clip = nullptr;        // ring of clipping factors by call, or null
  int clip_slots = 0;
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
  for (Chunk& c : t->chunks) {
    for (TcPlan* p : {c.factors, c.fwd1, c.adam, c.back1, c.wwrite}) tc_plan_destroy(p);
    destroy(c.rx);
    for (RxPlans& r : c.rx_layer) destroy(r);
  }
  for (TcPlan* p : t->factor_plan) tc_plan_destroy(p);
  delete t;
}

TcStep* tc_step_create(std::vector<Layer>& layers, const br_hparams& hp, char* scratch, size_t bytes,
                       const float* clip, int clip_slots, int device, cudaStream_t s, const char** err) {
  static thread_local std::string last;
  if (err) *err = nullptr;
  auto chunk_ids = make_chunks(layers, hp);
  if (chunk_ids.empty()) return nullptr;
  auto fail = [&](TcStep* t, const std::string& m) -> TcStep* {
    last = m; if (err) *err = last.c_str(); tc_step_destroy(t); return nullptr;
  };
  if (!tc_supported(device)) { last = "tensor-core path needs an sm_100 device and cuTensorMapEncodeTiled"; if (err) *err = last.c_str(); return nullptr; }
  TcStep* t = new TcStep();
  t->clip = clip; t->clip_slots = clip_slots;
  t->factor_plan.assign(layers.size(), nullptr);
  t->chunk_of.assign(layers.size(), -1);
  t->slot_of.assign(layers.size(), -1);
  const float beta_f = hp.beta_factor < 0.f ? hp.beta2 : hp.beta_factor;
  const char* perr = nullptr;
  auto build = [&](std::vector<TcProblem>& v, TcPlan** dst) -> bool {
    if (v.empty()) return true;
    *dst = tc_plan_create(v.data(), (int)v.size(), device, s, &perr);
    return *dst != nullptr;
  };
  for (const auto& ids : chunk_ids) {
    t->chunks.emplace_back();
    Chunk& c = t->chunks.back();
    c.ids = ids;
    size_t off = 0;
    auto take = [&](size_t numel) {
      __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(scratch + off);
      off += align_up(numel * 2);
      return p;
    };
    StepProblems P;
    RxProblems R;
    c.rx_layer.resize(ids.size());
    for (size_t j = 0; j < ids.size(); ++j) {
      const Layer& L = layers[ids[j]];
      t->chunk_of[ids[j]] = (int)t->chunks.size() - 1;
      t->slot_of[ids[j]] = (int)j;
      const int64_t mn = L.d.m * L.d.n;
      LayerScratch S;
      const int nb = (L.left && L.right) ? 4 : 2;
      for (int b = 0; b < nb; ++b) S.B[b] = take(mn);
      c.scr.push_back(S);
      if (off > bytes) return fail(t, "tensor-core scratch is smaller than the plan needs");
      if (L.d.src == BR_SRC_SECOND && hp.accum == BR_ACCUM_EVERY_STEP) factor_problems(L, beta_f, &P.factors);
      step_problems(L, S, hp, &P);
      rx_problems(L, S, &R);
      RxProblems one;
      rx_problems(L, S, &one);
      RxPlans& r = c.rx_layer[j];
      if (!build(one.back1, &r.back1) || !build(one.back2, &r.back2) || !build(one.fwd1, &r.fwd1) ||
          !build(one.fwd2, &r.fwd2))
        return fail(t, perr ? perr : "plan creation failed");
    }
    if (clip) {
      for (TcProblem& q : P.factors) { q.clip = clip; q.clip_slots = clip_slots; q.clip_mode = 2; }
      for (TcProblem& q : P.adam) { q.clip = clip; q.clip_slots = clip_slots; q.clip_mode = 1; }
    }
    if (!build(P.factors, &c.factors) || !build(P.fwd1, &c.fwd1) || !build(P.adam, &c.adam) ||
        !build(P.back1, &c.back1) || !build(P.wwrite, &c.wwrite) || !build(R.back1, &c.rx.back1) ||
        !build(R.back2, &c.rx.back2) || !build(R.fwd1, &c.rx.fwd1) || !build(R.fwd2, &c.rx.fwd2))
      return fail(t, perr ? perr : "plan creation failed");
  }
  if (hp.accum == BR_ACCUM_ON_REFRESH) {
    for (size_t i = 0; i < layers.size(); ++i) {
      const Layer& L = layers[i];
      if (!L.use_tc || L.d.src != BR_SRC_SECOND) continue;
      std::vector<TcProblem> f;
      factor_problems(L, beta_f, &f);
      if (clip) for (TcProblem& q : f) { q.clip = clip; q.clip_slots = clip_slots; q.clip_mode = 2; }
      if (!f.empty() && !(t->factor_plan[i] = tc_plan_create(f.data(), (int)f.size(), device, s, &perr)))
        return fail(t, perr ? perr : "plan creation failed");
    }
  }
  return t;
}

namespace {

struct Launcher {
  int* d_status; cudaStream_t s; LaunchStats* stats; const char** err;
  int fail(const char* what, cudaError_t e) {
    static thread_local std::string last;
    last = std::string(what) + ": " + cudaGetErrorString(e);
    if (err) *err = last.c_str();
    return (int)BR_ERR_CUDA;
  }
  int run(TcPlan* p, const char* what, long long calls, int tau, float a, float b) {
    if (!p) return 0;
    if (stats->inject()) return fail(what, cudaErrorLaunchFailure);     // host-side fault injection: nothing is launched
    const int span = stats->prof.begin(PROF_TC, s);
    cudaError_t e = tc_plan_launch(p, calls, tau, a, b, d_status, s);
    stats->prof.end(span, s, tc_plan_flops(p));
    if (e != cudaSuccess) return fail(what, e);
    stats->launches += 1;
    stats->gemm_flops += tc_plan_flops(p);
    return 0;
  }
  // re-expression plans read no ring and skip no layer: calls = 1, tau = 0 makes every problem active
  int run_rx(TcPlan* p, const char* what) { return run(p, what, 1, 0, 1.f, 0.f); }
};

// One direction of the re-expression for the layers at the given positions of chunk c.
int reexpress_chunk(Chunk& c, std::vector<Layer>& layers, const std::vector<int>& slots, bool forward,
                    Launcher& lz) {
  for (int j : slots) {
    const Layer& L = layers[c.ids[j]];
    cudaError_t e = split_bf16(L.M, c.scr[j].B[0], c.scr[j].B[1], L.d.m * L.d.n, lz.s);
    if (e != cudaSuccess) return lz.fail("split_bf16", e);
    lz.stats->launches += 1;
  }
  int rc;
  if (slots.size() == c.ids.size()) {
    if ((rc = lz.run_rx(forward ? c.rx.fwd1 : c.rx.back1, "re-expression, first side"))) return rc;
    if ((rc = lz.run_rx(forward ? c.rx.fwd2 : c.rx.back2, "re-expression, second side"))) return rc;
  } else {
    for (int j : slots) {
      RxPlans& r = c.rx_layer[j];
      if ((rc = lz.run_rx(forward ? r.fwd1 : r.back1, "re-expression, first side"))) return rc;
      if ((rc = lz.run_rx(forward ? r.fwd2 : r.back2, "re-expression, second side"))) return rc;
    }
  }
  return 0;
}

}  // namespace

int tc_step_reexpress(TcStep* t, std::vector<Layer>& layers, const int* ids, int n, int forward, int* d_status,
                      cudaStream_t s, LaunchStats* stats, const char** err) {
  if (!t) return 0;
  Launcher lz{d_status, s, stats, err};
  for (size_t ci = 0; ci < t->chunks.size(); ++ci) {
    std::vector<int> slots;
    for (int k = 0; k < n; ++k)
      if (ids[k] >= 0 && ids[k] < (int)layers.size() && t->chunk_of[ids[k]] == (int)ci) slots.push_back(t->slot_of[ids[k]]);
    if (slots.empty()) continue;
    std::sort(slots.begin(), slots.end());
    int rc = reexpress_chunk(t->chunks[ci], layers, slots, forward != 0, lz);
    if (rc) return rc;
  }
  return 0;
}

int tc_step_run(TcStep* t, std::vector<Layer>& layers, const std::vector<const void*>& G, long long calls,
                int tau, const br_hparams& hp, int* d_status, cudaStream_t s, LaunchStats* stats,
                const TcStepCallbacks& cb, const char** err) {
  Launcher lz{d_status, s, stats, err};
  const float dyn_alpha = -hp.lr, dyn_beta = 1.0f - hp.lr * hp.weight_decay;
  for (Chunk& c : t->chunks) {
    bool any = false;
    for (int i : c.ids) any = any || G[i] != nullptr;
    if (!any) continue;
    int rc;
    if ((rc = lz.run(c.factors, "factor launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
    if (c.factors)
      for (int i : c.ids) if (G[i]) layers[i].n_accum += 1;
    std::vector<int> due, due_slots;
    for (size_t j = 0; j < c.ids.size(); ++j) {
      const int i = c.ids[j];
      Layer& L = layers[i];
      if (!G[i] || L.t % L.freq != 0) continue;
      if (t->factor_plan[i]) {
        if ((rc = lz.run(t->factor_plan[i], "factor launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
        L.n_accum += 1;
      }
      due.push_back(i);
      due_slots.push_back((int)j);
    }
    if (!due.empty()) {
      // M_{t-1} = U M~_{t-1} V^T with the old basis; S = 1st refreshes from M_t = b1 M_{t-1} + (1-b1) G
      if ((rc = reexpress_chunk(c, layers, due_slots, false, lz))) return rc;
      for (int i : due) {
        Layer& L = layers[i];
        if (L.d.src != BR_SRC_FIRST) continue;
        const int tl = tau < 0 ? L.d.tau_max : tau;
        const float* gs = t->clip ? t->clip + (int)((calls - 1 - tl) % t->clip_slots) : nullptr;
        cudaError_t e = ema_out(L.Morig, L.M, G[i], L.d.grad_dtype == BR_BF16, L.d.m * L.d.n, hp.beta1, gs, s);
        if (e != cudaSuccess) return lz.fail("ema_out", e);
        stats->launches += 1;
      }
      rc = cb.refresh(cb.ctx, due.data(), (int)due.size());
      if (rc != 0) { if (err) *err = nullptr; return rc; }
      // M~_{t-1} = U^T M_{t-1} V with the new basis
      if ((rc = reexpress_chunk(c, layers, due_slots, true, lz))) return rc;
    }
    if ((rc = lz.run(c.fwd1, "first-side rotation launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
    if ((rc = lz.run(c.adam, "rotated-Adam launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
    if (cb.consumed) {       // factors, first side and (one-sided layers) rotated Adam were the readers of G
      rc = cb.consumed(cb.ctx, c.ids.data(), (int)c.ids.size());
      if (rc != 0) { if (err) *err = nullptr; return rc; }
    }
    if ((rc = lz.run(c.back1, "back-rotation launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
    if ((rc = lz.run(c.wwrite, "weight-write launch", calls, tau, dyn_alpha, dyn_beta))) return rc;
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
