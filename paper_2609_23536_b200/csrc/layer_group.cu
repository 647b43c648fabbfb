// Layer API, several actions per call: grouped weight gradients, chained linears with FP8 hand-off, independent
// actions in shared launches (pairs, qe_run_together) and the whole-step call with its round planner.
#include "layer_impl.h"

using namespace qe_impl;

extern "C" {

int32_t qe_backward_dW_multi(qe_layer* const* layers, const qe_tape* tapes, uint32_t n, float* grad, uint64_t elems,
                             const uint64_t* offsets, void* caller_stream) {
  if (!layers || !tapes || !offsets || n == 0 || n > QE_MAX_MULTI_DW) return fail(QE_ERR_BAD_ARG, "null argument or bad count %u", n);
  qe_ctx* ctx = layers[0] ? layers[0]->ctx : nullptr;
  for (uint32_t i = 0; i < n; ++i) {
    if (!layers[i] || layers[i]->ctx != ctx) return fail(QE_ERR_BAD_ARG, "layer %u is null or belongs to another context", i);
    for (uint32_t j = 0; j < i; ++j)
      if (layers[j] == layers[i]) return fail(QE_ERR_BAD_ARG, "layer %u appears twice", i);
  }
  // check (every layer, before anything runs) -> run -> commit
  int32_t acc[QE_MAX_MULTI_DW];
  int32_t st;
  for (uint32_t i = 0; i < n; ++i) {
    const uint64_t slice = (uint64_t)layers[i]->cfg.N * layers[i]->cfg.K;
    if ((st = qe_contract_dW_check(layers[i]->contract, &tapes[i], (uint64_t)(uintptr_t)grad, elems, offsets[i], slice, &acc[i])) != QE_OK)
      return st;
  }
  cudaStream_t caller = (cudaStream_t)caller_stream;
  cudaStream_t run_on = ctx->exec_stream;
  if (ctx->dw_stream) {
    run_on = ctx->dw_stream;
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, caller));
    QE_CUDA(cudaStreamWaitEvent(run_on, ctx->ev_dw_in, 0));
    for (uint32_t i = 0; i < n; ++i) QE_CUDA(cudaStreamWaitEvent(run_on, layers[i]->ev_di[tapes[i].ref.slot], 0));
    ctx->stats.handoffs += 1;
  } else if ((st = handoff_in(ctx, caller)) != QE_OK) {
    return st;
  }
  std::vector<qe::Launch> ls;
  DWBatch dwb;
  Fnv h;
  h.mix("dWmulti", 8);
  for (uint32_t i = 0; i < n; ++i) {
    const uint32_t p = tapes[i].ref.slot;
    dwb.add(ctx, layers[i], dW_gemm(layers[i], p, grad + offsets[i], acc[i], nullptr), ls);
    h.mix(&layers[i], sizeof(qe_layer*));
    h.mix(&p, sizeof(p));
  }
  dwb.flush(ctx, ls);
  if (ctx->exec_mode == QE_EXEC_GRAPH) {
    ActionGraph* g = keyed_graph(ctx, h.key, ls.size());
    if (!g) return fail(QE_ERR_BAD_ARG, "out of host memory");
    st = run_action(ctx, g, ls, run_on);
  } else {
    for (const qe::Launch& l : ls)
      if ((st = launch_eager(ctx, l, run_on)) != QE_OK) break;
  }
  if (st != QE_OK) return st;
  if (ctx->dw_stream) {
    for (uint32_t i = 0; i < n; ++i) {
      const uint32_t p = tapes[i].ref.slot;
      QE_CUDA(cudaEventRecord(layers[i]->ev_dw[p], run_on));
      layers[i]->dw_pending[p] = true;
    }
  } else if ((st = handoff_out(ctx, caller)) != QE_OK) {
    return st;
  }
  for (uint32_t i = 0; i < n; ++i) {
    const uint64_t slice = (uint64_t)layers[i]->cfg.N * layers[i]->cfg.K;
    if ((st = qe_contract_dW_commit(layers[i]->contract, &tapes[i], (uint64_t)(uintptr_t)grad, offsets[i], slice)) != QE_OK) return st;
  }
  return QE_OK;
}

// ------------------------------------------------------------------------------------------------ chained linears
static int32_t check_chain(qe_layer* const* layers, uint32_t n) {
  if (!layers || n == 0 || n > QE_MAX_CHAIN) return fail(QE_ERR_BAD_ARG, "null argument or bad chain length %u", n);
  for (uint32_t i = 0; i < n; ++i) {
    if (!layers[i] || layers[i]->ctx != layers[0]->ctx) return fail(QE_ERR_BAD_ARG, "layer %u is null or belongs to another context", i);
    for (uint32_t j = 0; j < i; ++j)
      if (layers[j] == layers[i]) return fail(QE_ERR_BAD_ARG, "layer %u appears twice", i);
    if (i && (layers[i]->cfg.T != layers[0]->cfg.T || layers[i]->cfg.K != layers[i - 1]->cfg.N))
      return fail(QE_ERR_SHAPE, "layer %u does not take layer %u's output ([%u, %u] after [%u, %u])", i, i - 1, layers[i]->cfg.T,
                  layers[i]->cfg.K, layers[i - 1]->cfg.T, layers[i - 1]->cfg.N);
  }
  // a deposited FP8 tensor is the row-major one only: every layer that receives one must run without transposed copies
  for (uint32_t i = 0; i < n; ++i)
    if ((i > 0 && layers[i]->XqT[0]) || (i + 1 < n && layers[i]->GqT[0]))
      return fail(QE_ERR_UNSUPPORTED, "layer %u keeps transposed FP8 copies (T and N must be multiples of 256 for the hand-off)", i);
  return QE_OK;
}

int32_t qe_forward_chain(qe_layer* const* layers, uint32_t n, uint32_t mb, uint64_t gen, const void* x, void* y,
                         void* caller_stream, qe_tape* tapes_out) {
  int32_t st = check_chain(layers, n);
  if (st != QE_OK) return st;
  if (!x || !y || !tapes_out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (((uintptr_t)x | (uintptr_t)y) & 15u) return fail(QE_ERR_BAD_ARG, "x and y must be 16-byte aligned");
  int32_t refresh[QE_MAX_CHAIN];
  uint32_t p[QE_MAX_CHAIN];
  for (uint32_t i = 0; i < n; ++i)  // every layer's check before anything runs
    if ((st = qe_contract_forward_check(layers[i]->contract, mb, gen, &refresh[i], &p[i])) != QE_OK) return st;
  qe_ctx* ctx = layers[0]->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  std::vector<qe::Launch> ls;
  Fnv h;
  h.mix("Fchain", 7);
  for (uint32_t i = 0; i < n; ++i) {
    qe_layer* L = layers[i];
    if (L->dw_pending[p[i]]) {
      QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, L->ev_dw[p[i]], 0));
      L->dw_pending[p[i]] = false;
    }
    if (refresh[i]) add_refresh(L, ls);
    h.mix(&layers[i], sizeof(qe_layer*));
    h.mix(&p[i], sizeof(uint32_t));
    h.mix(&refresh[i], sizeof(int32_t));
  }
  for (uint32_t i = 0; i < n; ++i) {
    const bool last = i + 1 == n;
    add_forward(layers[i], p[i], i == 0 ? x : nullptr, last ? y : nullptr, ls, last ? nullptr : layers[i + 1], last ? 0 : p[i + 1]);
  }
  if ((st = run_keyed(ctx, h.key, ls)) != QE_OK) return st;
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  for (uint32_t i = 0; i < n; ++i)
    if ((st = qe_contract_forward_commit(layers[i]->contract, mb, &tapes_out[i])) != QE_OK) return st;
  return QE_OK;
}

int32_t qe_backward_dI_chain(qe_layer* const* layers, const qe_tape* tapes, uint32_t n, const void* dy, void* dx,
                             void* caller_stream) {
  int32_t st = check_chain(layers, n);
  if (st != QE_OK) return st;
  if (!tapes || !dy || !dx) return fail(QE_ERR_BAD_ARG, "null argument");
  if (((uintptr_t)dy | (uintptr_t)dx) & 15u) return fail(QE_ERR_BAD_ARG, "dy and dx must be 16-byte aligned");
  for (uint32_t i = 0; i < n; ++i)
    if ((st = qe_contract_dI_check(layers[i]->contract, &tapes[i])) != QE_OK) return st;
  qe_ctx* ctx = layers[0]->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  std::vector<qe::Launch> ls;
  Fnv h;
  h.mix("Bchain", 7);
  for (uint32_t k = n; k-- > 0;) {  // last linear first
    const uint32_t pk = tapes[k].ref.slot;
    add_dI(layers[k], pk, k + 1 == n ? dy : nullptr, k == 0 ? dx : nullptr, ls, k ? layers[k - 1] : nullptr,
           k ? tapes[k - 1].ref.slot : 0);
    h.mix(&layers[k], sizeof(qe_layer*));
    h.mix(&pk, sizeof(uint32_t));
  }
  if ((st = run_keyed(ctx, h.key, ls)) != QE_OK) return st;
  if (ctx->dw_stream)
    for (uint32_t i = 0; i < n; ++i) QE_CUDA(cudaEventRecord(layers[i]->ev_di[tapes[i].ref.slot], ctx->exec_stream));
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  for (uint32_t i = 0; i < n; ++i)
    if ((st = qe_contract_dI_commit(layers[i]->contract, &tapes[i])) != QE_OK) return st;
  return QE_OK;
}

// ------------------------------------------------------------------------------------------------ F and dI together
// In the steady state of a split-backward schedule a stage holds a forward unit (microbatch m + k) and an input-
// gradient unit (microbatch m) at the same time.  Their chains through the layers are independent, so F of layer i
// and dI of layer j (two different layers) can share one GEMM launch: one fixed cost and common waves.
int32_t qe_forward_dI_pair(qe_layer* Lf, uint32_t mb, uint64_t gen, const void* x, void* y, qe_tape* tape_out,
                           qe_layer* Lb, const qe_tape* tape_b, const void* dy, void* dx, void* caller_stream) {
  if (!Lf || !Lb || !x || !y || !tape_out || !tape_b || !dy || !dx) return fail(QE_ERR_BAD_ARG, "null argument");
  if (Lf == Lb || Lf->ctx != Lb->ctx) return fail(QE_ERR_BAD_ARG, "the two layers must be different layers of one context");
  if (((uintptr_t)x | (uintptr_t)y | (uintptr_t)dy | (uintptr_t)dx) & 15u) return fail(QE_ERR_BAD_ARG, "tensors must be 16-byte aligned");
  int32_t refresh = 0;
  uint32_t p = 0;
  int32_t st = qe_contract_forward_check(Lf->contract, mb, gen, &refresh, &p);  // both checks before anything runs
  if (st != QE_OK) return st;
  if ((st = qe_contract_dI_check(Lb->contract, tape_b)) != QE_OK) return st;
  qe_ctx* ctx = Lf->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  const uint32_t pb = tape_b->ref.slot;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  if (Lf->dw_pending[p]) {
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, Lf->ev_dw[p], 0));
    Lf->dw_pending[p] = false;
  }
  std::vector<qe::Launch> ls;
  if (refresh) add_refresh(Lf, ls);
  qe::GemmParams g[2];
  qe::QuantParams c[2];
  add_forward(Lf, p, x, y, ls, nullptr, 0, &g[0], &c[0]);  // hands the casts and the GEMMs back
  add_dI(Lb, pb, dy, dx, ls, nullptr, 0, &g[1], &c[1]);
  ls.push_back(qe::make_quantize_multi(c, 2));  // both casts in one launch
  qe::Launch shared;
  if (qe::make_gemm_group(g, 2, ctx->dev->num_sms, &shared)) {
    ls.push_back(shared);
    ctx->stats.paired_f_di += 1;
  } else {  // a shape that needs the single-CTA variant: one after the other
    ls.push_back(qe::make_gemm(g[0], ctx->dev->num_sms));
    ls.push_back(qe::make_gemm(g[1], ctx->dev->num_sms));
  }
  Fnv h;
  h.mix("FdI", 4);
  h.mix(&Lf, sizeof(Lf));
  h.mix(&Lb, sizeof(Lb));
  h.mix(&p, sizeof(p));
  h.mix(&pb, sizeof(pb));
  h.mix(&refresh, sizeof(refresh));
  if ((st = run_keyed(ctx, h.key, ls)) != QE_OK) return st;
  if (ctx->dw_stream) QE_CUDA(cudaEventRecord(Lb->ev_di[pb], ctx->exec_stream));
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  if ((st = qe_contract_forward_commit(Lf->contract, mb, tape_out)) != QE_OK) return st;
  return qe_contract_dI_commit(Lb->contract, tape_b);
}

// ------------------------------------------------------------------------------------------------ independent actions
namespace {
struct TogetherPrep {
  int32_t refresh[QE_MAX_TOGETHER] = {}, acc[QE_MAX_TOGETHER] = {};
  uint32_t slot[QE_MAX_TOGETHER] = {};
  bool any_dw = false;
};

// argument rules and every action's contract check; nothing is changed
int32_t together_prepare(qe_ctx* ctx, const qe_action* acts, uint32_t n, float* grad, uint64_t grad_elems, TogetherPrep* pr) {
  if (!ctx || !acts || n == 0 || n > QE_MAX_TOGETHER) return fail(QE_ERR_BAD_ARG, "null argument or bad count %u", n);
  for (uint32_t i = 0; i < n; ++i) {
    const qe_action& a = acts[i];
    if (a.kind > QE_ACT_DW || !a.layer || a.layer->ctx != ctx || !a.tape) return fail(QE_ERR_BAD_ARG, "action %u: bad kind, layer or tape", i);
    if (a.kind != QE_ACT_DW && (!a.in_dev || !a.out_dev || (((uintptr_t)a.in_dev | (uintptr_t)a.out_dev) & 15u)))
      return fail(QE_ERR_BAD_ARG, "action %u: input / output null or misaligned", i);
    for (uint32_t j = 0; j < i; ++j)
      if (acts[j].layer == a.layer && acts[j].kind == a.kind) return fail(QE_ERR_BAD_ARG, "actions %u and %u: same kind on the same layer", j, i);
    pr->any_dw |= a.kind == QE_ACT_DW;
  }
  if (pr->any_dw && !grad) return fail(QE_ERR_BAD_ARG, "gradient buffer is null");
  for (uint32_t i = 0; i < n; ++i) {
    const qe_action& a = acts[i];
    qe_layer* L = a.layer;
    int32_t st;
    if (a.kind == QE_ACT_F) {
      st = qe_contract_forward_check(L->contract, a.mb, a.gen, &pr->refresh[i], &pr->slot[i]);
    } else if (a.kind == QE_ACT_DI) {
      st = qe_contract_dI_check(L->contract, a.tape);
      pr->slot[i] = a.tape->ref.slot;
    } else {
      st = qe_contract_dW_check(L->contract, a.tape, (uint64_t)(uintptr_t)grad, grad_elems, a.grad_offset, (uint64_t)L->cfg.N * L->cfg.K, &pr->acc[i]);
      pr->slot[i] = a.tape->ref.slot;
    }
    if (st != QE_OK) return st;
  }
  return QE_OK;
}

// the launches: the casts in one launch, then every GEMM that can run on the paired variant in one launch
int32_t together_build(qe_ctx* ctx, const qe_action* acts, uint32_t n, const TogetherPrep& pr, float* grad,
                       std::vector<qe::Launch>& ls, Fnv* h) {
  qe::GemmParams g[QE_MAX_TOGETHER];
  qe::QuantParams casts[QE_MAX_TOGETHER];
  std::vector<qe::GemmParams> singles;
  uint32_t ng = 0, n_chain = 0, n_dw = 0, n_casts = 0;
  for (int pass = 0; pass < 2; ++pass) {  // F and dI first (others wait for them), the weight gradients' tiles after theirs
    for (uint32_t i = 0; i < n; ++i) {
      const qe_action& a = acts[i];
      qe_layer* L = a.layer;
      if ((a.kind == QE_ACT_DW) != (pass == 1)) continue;
      qe::GemmParams gp;
      if (a.kind == QE_ACT_F) {
        if (L->dw_pending[pr.slot[i]]) {
          QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, L->ev_dw[pr.slot[i]], 0));
          L->dw_pending[pr.slot[i]] = false;
        }
        if (pr.refresh[i]) add_refresh(L, ls);
        add_forward(L, pr.slot[i], a.in_dev, a.out_dev, ls, nullptr, 0, &gp, &casts[n_casts++]);
      } else if (a.kind == QE_ACT_DI) {
        add_dI(L, pr.slot[i], a.in_dev, a.out_dev, ls, nullptr, 0, &gp, &casts[n_casts++]);
      } else {
        gp = dW_gemm(L, pr.slot[i], grad + a.grad_offset, pr.acc[i], nullptr);
      }
      if (qe::gemm_uses_pair(gp.M)) {
        g[ng++] = gp;
        (a.kind == QE_ACT_DW ? n_dw : n_chain) += 1;
      } else {
        singles.push_back(gp);  // single-CTA variant: a launch of its own
      }
      if (h) {
        h->mix(&a.kind, sizeof(a.kind));
        h->mix(&a.layer, sizeof(a.layer));
        h->mix(&pr.slot[i], sizeof(uint32_t));
        h->mix(&pr.refresh[i], sizeof(int32_t));
      }
    }
  }
  // longest tiles first (their contraction length decides a tile's duration): the launch's last, partial wave is then
  // made of short tiles.  The weight gradients (contraction over T only) stay behind the others.
  std::stable_sort(g, g + n_chain, [](const qe::GemmParams& x, const qe::GemmParams& y) { return x.Kc > y.Kc; });
  std::stable_sort(g + n_chain, g + ng, [](const qe::GemmParams& x, const qe::GemmParams& y) { return x.Kc > y.Kc; });
  if (n_casts >= 2) ls.push_back(qe::make_quantize_multi(casts, n_casts));  // all casts of the call in one launch
  else if (n_casts == 1) ls.push_back(qe::make_quantize(casts[0]));
  for (const qe::GemmParams& gp : singles) ls.push_back(qe::make_gemm(gp, ctx->dev->num_sms));
  qe::Launch shared;
  if (ng >= 2 && qe::make_gemm_group(g, ng, ctx->dev->num_sms, &shared)) {
    ls.push_back(shared);
    ctx->stats.grouped_dw += n_dw;
    ctx->stats.paired_f_di += n_chain >= 1 ? 1 : 0;
  } else {
    for (uint32_t i = 0; i < ng; ++i) ls.push_back(qe::make_gemm(g[i], ctx->dev->num_sms));
  }
  return QE_OK;
}

// Forward commits first: a forward's tape slot was chosen by its check, on the state before the call, and the kernels
// used it; a weight-gradient commit of the same layer releases a slot and must not come in between.
int32_t together_commit(const qe_action* acts, uint32_t n, float* grad, const TogetherPrep& pr) {
  for (uint32_t kind = QE_ACT_F; kind <= QE_ACT_DW; ++kind) {
    for (uint32_t i = 0; i < n; ++i) {
      const qe_action& a = acts[i];
      if (a.kind != kind) continue;
      qe_layer* L = a.layer;
      int32_t st;
      if (a.kind == QE_ACT_F) {
        st = qe_contract_forward_commit(L->contract, a.mb, a.tape);
        if (st == QE_OK && a.tape->ref.slot != pr.slot[i]) return fail(QE_ERR_ORDER, "forward committed to slot %u, ran in slot %u", a.tape->ref.slot, pr.slot[i]);
      } else if (a.kind == QE_ACT_DI) {
        st = qe_contract_dI_commit(L->contract, a.tape);
      } else {
        st = qe_contract_dW_commit(L->contract, a.tape, (uint64_t)(uintptr_t)grad, a.grad_offset, (uint64_t)L->cfg.N * L->cfg.K);
      }
      if (st != QE_OK) return st;
    }
  }
  return QE_OK;
}
}  // namespace

// host != 0: the in / out pointers of the F and dI actions are HOST buffers, staged through the layers' fixed device
// buffers like qe_forward_host / qe_backward_dI_host do (uploads of all actions first, read-backs after the kernels).
static int32_t run_together_impl(qe_ctx* ctx, qe_action* acts, uint32_t n, float* grad, uint64_t grad_elems, void* caller_stream,
                                 int host) {
  if (!ctx || !acts || n == 0 || n > QE_MAX_TOGETHER) return fail(QE_ERR_BAD_ARG, "null argument or bad count %u", n);
  qe_action dev[QE_MAX_TOGETHER];
  for (uint32_t i = 0; i < n; ++i) {
    dev[i] = acts[i];
    if (!host || acts[i].kind > QE_ACT_DI || !acts[i].layer) continue;
    qe_layer* L = acts[i].layer;
    if (!L->x_stage) return fail(QE_ERR_BAD_ARG, "action %u: layer was created without host_io", i);
    if (!acts[i].in_dev) return fail(QE_ERR_BAD_ARG, "action %u: host input is null", i);
    dev[i].in_dev = acts[i].kind == QE_ACT_F ? L->x_stage : L->dy_stage;
    dev[i].out_dev = acts[i].kind == QE_ACT_F ? L->y_stage : L->dx_stage;
  }
  TogetherPrep pr;
  int32_t st = together_prepare(ctx, dev, n, grad, grad_elems, &pr);  // check (every action, before anything runs)
  if (st != QE_OK) return st;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  if (host)
    for (uint32_t i = 0; i < n; ++i) {
      if (acts[i].kind > QE_ACT_DI) continue;
      const qe_layer_config& c = acts[i].layer->cfg;
      const size_t bytes = 2ull * c.T * (acts[i].kind == QE_ACT_F ? c.K : c.N);
      if ((st = host_upload(ctx, const_cast<void*>(dev[i].in_dev), acts[i].in_dev, bytes, caller)) != QE_OK) return st;
    }
  if (pr.any_dw && ctx->dw_stream) {  // weight gradients issued earlier on the second stream accumulate into the same buffer
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, ctx->dw_stream));
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_dw_in, 0));
  }
  std::vector<qe::Launch> ls;
  Fnv h;
  h.mix("together", 9);
  if ((st = together_build(ctx, dev, n, pr, grad, ls, &h)) != QE_OK) return st;
  if ((st = run_keyed(ctx, h.key, ls)) != QE_OK) return st;  // ... run ...
  if (host)
    for (uint32_t i = 0; i < n; ++i) {
      if (acts[i].kind > QE_ACT_DI) continue;
      const qe_layer_config& c = acts[i].layer->cfg;
      const size_t bytes = 2ull * c.T * (acts[i].kind == QE_ACT_F ? c.N : c.K);
      if ((st = host_download(ctx, acts[i].out_dev, dev[i].out_dev, bytes)) != QE_OK) return st;
    }
  if (ctx->dw_stream)
    for (uint32_t i = 0; i < n; ++i)
      if (acts[i].kind == QE_ACT_DI) QE_CUDA(cudaEventRecord(acts[i].layer->ev_di[pr.slot[i]], ctx->exec_stream));
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  return together_commit(dev, n, grad, pr);  // ... commit (the tapes are written through the callers' pointers)
}

int32_t qe_run_together(qe_ctx* ctx, qe_action* acts, uint32_t n, float* grad, uint64_t grad_elems, void* caller_stream) {
  return run_together_impl(ctx, acts, n, grad, grad_elems, caller_stream, 0);
}

int32_t qe_run_together_host(qe_ctx* ctx, qe_action* acts, uint32_t n, float* grad, uint64_t grad_elems, void* caller_stream) {
  return run_together_impl(ctx, acts, n, grad, grad_elems, caller_stream, 1);
}

// ------------------------------------------------------------------------------------------------ whole-step call
int32_t qe_step_run(qe_ctx* ctx, qe_layer* const* layers, uint32_t n_layers, const qe_step_action* actions,
                    uint32_t n_actions, uint32_t M, const qe_step_io* io, float* grad, uint64_t grad_elems,
                    const uint64_t* offsets, float* temp, void* caller_stream) {
  if (!ctx || !layers || !actions || !io || !offsets) return fail(QE_ERR_BAD_ARG, "null argument");
  if (n_layers == 0 || n_actions == 0 || M == 0 || M > QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "empty list or bad microbatch count");
  if (temp && ((uintptr_t)temp & 15u)) return fail(QE_ERR_BAD_ARG, "temp_dev must be 16-byte aligned");
  for (uint32_t l = 0; l < n_layers; ++l)
    if (!layers[l] || layers[l]->ctx != ctx) return fail(QE_ERR_BAD_ARG, "layer %u is null or belongs to another context", l);
  cudaStream_t caller = (cudaStream_t)caller_stream;

  std::vector<qe_tape> tapes((size_t)n_layers * M);
  std::vector<uint8_t> have((size_t)n_layers * M, 0);
  std::vector<qe::Launch> ls;
  ls.reserve(2 * (size_t)n_actions + n_layers);
  int32_t st = QE_OK;
  uint32_t k = 0;

  // ---- issue plan.  The list is read as units (runs of actions of one kind and microbatch over distinct layers: a
  // forward, input-gradient or weight-gradient unit of the stage).  Units a stage holds at the same time are
  // independent, so the list is cut into rounds of actions whose predecessors were issued in earlier rounds -- the
  // previous layer of the own unit (F and dI walk their layers in list order), the same layer of the previous unit of
  // the kind, F before dI before dW of a (layer, microbatch), a free tape slot -- looking `window` units ahead, and a
  // round goes out as qe_run_together would issue it.  If no such plan exists (an illegal list) the action-by-action
  // pass below runs instead and reports the failing action.
  std::vector<std::vector<uint32_t>> rounds;  // indices into actions[]
  if (!temp && ctx->step_window > 1) {
    std::vector<uint32_t> slots(n_layers), live(n_layers), round_of(n_actions);
    for (uint32_t l = 0; l < n_layers; ++l) {
      slots[l] = layers[l]->cfg.slots;
      live[l] = layers[l]->contract->live_tapes();
    }
    uint32_t n_rounds = 0;
    if (qe_plan_rounds(actions, n_actions, n_layers, M, slots.data(), live.data(), ctx->step_window, QE_MAX_TOGETHER,
                       round_of.data(), &n_rounds) == QE_OK) {
      rounds.resize(n_rounds);
      for (uint32_t i = 0; i < n_actions; ++i) rounds[round_of[i]].push_back(i);
    }
  }
  for (size_t r = 0; r < rounds.size() && st == QE_OK; ++r) {
    qe_action acts[QE_MAX_TOGETHER];
    uint32_t na = 0;
    for (uint32_t gi : rounds[r]) {
      const qe_step_action& a = actions[gi];
      const size_t u = (size_t)a.layer * M + a.mb;
      qe_layer* L = layers[a.layer];
      if (a.kind == QE_ACT_F) acts[na++] = qe_action{QE_ACT_F, a.mb, L->contract->e_W, L, io[u].x_dev, io[u].y_dev, &tapes[u], 0};
      else if (a.kind == QE_ACT_DI) acts[na++] = qe_action{QE_ACT_DI, 0, 0, L, io[u].dy_dev, io[u].dx_dev, &tapes[u], 0};
      else acts[na++] = qe_action{QE_ACT_DW, 0, 0, L, nullptr, nullptr, &tapes[u], offsets[a.layer]};
    }
    TogetherPrep pr;
    if ((st = together_prepare(ctx, acts, na, grad, grad_elems, &pr)) != QE_OK || (st = together_build(ctx, acts, na, pr, grad, ls, nullptr)) != QE_OK) {
      k = rounds[r][0];  // (reported as the index of the first action of the failing round)
      break;
    }
    st = together_commit(acts, na, grad, pr);
  }
  if (!rounds.empty()) k = st == QE_OK ? n_actions : k;

  // ---- host pass: check -> collect launches -> commit, action by action (Algorithm 1)
  DWBatch dwb;
  for (; rounds.empty() && k < n_actions && st == QE_OK; ++k) {
    const qe_step_action& a = actions[k];
    if (a.kind != QE_ACT_DW && dwb.n) dwb.flush(ctx, ls);
    if (a.layer >= n_layers || a.mb >= M || a.kind > QE_ACT_DW) {
      st = fail(QE_ERR_BAD_ARG, "action %u: kind %u layer %u mb %u", k, a.kind, a.layer, a.mb);
      break;
    }
    qe_layer* L = layers[a.layer];
    const size_t u = (size_t)a.layer * M + a.mb;
    const qe_step_io& b = io[u];
    if (a.kind == QE_ACT_F) {
      int32_t refresh = 0;
      uint32_t p = 0;
      if (!b.x_dev || !b.y_dev || (((uintptr_t)b.x_dev | (uintptr_t)b.y_dev) & 15u)) { st = fail(QE_ERR_BAD_ARG, "action %u: x/y null or misaligned", k); break; }
      if ((st = qe_contract_forward_check(L->contract, a.mb, L->contract->e_W, &refresh, &p)) != QE_OK) break;
      if (L->dw_pending[p]) {  // a dW issued earlier through the overlapped per-action path still reads this slot
        cudaStreamWaitEvent(ctx->exec_stream, L->ev_dw[p], 0);
        L->dw_pending[p] = false;
      }
      if (refresh) add_refresh(L, ls);
      add_forward(L, p, b.x_dev, b.y_dev, ls);
      st = qe_contract_forward_commit(L->contract, a.mb, &tapes[u]);
      have[u] = 1;
    } else if (a.kind == QE_ACT_DI) {
      if (!have[u]) { st = fail(QE_ERR_ORDER, "action %u: dI before F in this list", k); break; }
      if (!b.dy_dev || !b.dx_dev || (((uintptr_t)b.dy_dev | (uintptr_t)b.dx_dev) & 15u)) { st = fail(QE_ERR_BAD_ARG, "action %u: dy/dx null or misaligned", k); break; }
      if ((st = qe_contract_dI_check(L->contract, &tapes[u])) != QE_OK) break;
      add_dI(L, tapes[u].ref.slot, b.dy_dev, b.dx_dev, ls);
      st = qe_contract_dI_commit(L->contract, &tapes[u]);
    } else {
      if (!have[u]) { st = fail(QE_ERR_ORDER, "action %u: dW before F in this list", k); break; }
      const uint64_t slice = (uint64_t)L->cfg.N * L->cfg.K;
      int32_t acc = 0;
      if ((st = qe_contract_dW_check(L->contract, &tapes[u], (uint64_t)(uintptr_t)grad, grad_elems, offsets[a.layer], slice, &acc)) != QE_OK) break;
      if (temp) add_dW(L, tapes[u].ref.slot, grad + offsets[a.layer], acc, temp, ls);
      else dwb.add(ctx, L, dW_gemm(L, tapes[u].ref.slot, grad + offsets[a.layer], acc, nullptr), ls);
      st = qe_contract_dW_commit(L->contract, &tapes[u], (uint64_t)(uintptr_t)grad, offsets[a.layer], slice);
    }
  }
  if (dwb.n) dwb.flush(ctx, ls);
  const int32_t check_status = st;
  char saved_msg[512];
  std::snprintf(saved_msg, sizeof(saved_msg), "%s", qe_last_error());

  // ---- device pass: the launches of every action that passed, behind one handshake
  int32_t run_status = QE_OK;
  if (!ls.empty()) {
    run_status = handoff_in(ctx, caller);
    if (run_status == QE_OK && ctx->dw_stream) {
      // weight-gradient work issued earlier through the overlapped per-action path must finish first: this list's
      // dW kernels run on the execution stream and accumulate into the same buffer
      cudaError_t e = cudaEventRecord(ctx->ev_dw_in, ctx->dw_stream);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_dw_in, 0);
      if (e != cudaSuccess) run_status = fail(QE_ERR_CUDA, "joining the dW stream: %s", cudaGetErrorString(e));
    }
    if (run_status == QE_OK) {
      if (ctx->exec_mode == QE_EXEC_GRAPH && check_status == QE_OK) {
        Fnv h;  // over the list's identity
        h.mix(layers, sizeof(qe_layer*) * n_layers);
        h.mix(actions, sizeof(qe_step_action) * n_actions);
        h.mix(&M, sizeof(M));
        ActionGraph* g = keyed_graph(ctx, h.key, ls.size());
        if (!g) return fail(QE_ERR_BAD_ARG, "out of host memory");
        run_status = run_action(ctx, g, ls);
      } else {
        for (const qe::Launch& l : ls)
          if ((run_status = launch_eager(ctx, l, ctx->exec_stream)) != QE_OK) break;
      }
    }
    if (run_status == QE_OK) run_status = handoff_out(ctx, caller);
  }
  if (check_status != QE_OK || run_status != QE_OK) {
    // failure boundary: outstanding tapes aborted, arenas unusable for the epoch
    for (uint32_t l = 0; l < n_layers; ++l) qe_contract_abort(layers[l]->contract);
    if (check_status != QE_OK) return fail(check_status, "step aborted at action %u: %s", k, saved_msg);
    return run_status;
  }
  return QE_OK;
}

}  // extern "C"
