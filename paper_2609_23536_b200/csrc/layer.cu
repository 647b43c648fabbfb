// Layer API, one action per call: context and layer objects, F / dI / dW (device and host buffers, staged and arena
// variants), boundary, scale commit, abort / rebuild, state views and checkpoints.
#include "layer_impl.h"

using namespace qe_impl;

extern "C" {

int32_t qe_ctx_create(const qe_ctx_config* cfg, qe_ctx** out) {
  if (!cfg || !out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (cfg->exec_mode > QE_EXEC_GRAPH) return fail(QE_ERR_BAD_ARG, "exec_mode %u", cfg->exec_mode);
  if (cfg->flags & ~(QE_CTX_OVERLAP_DW | QE_CTX_UNSAFE_ONE_WAY_HANDOFF)) return fail(QE_ERR_BAD_ARG, "unknown flags %#x", cfg->flags);
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev == 0) return fail(QE_ERR_UNSUPPORTED, "no CUDA device: %s", cudaGetErrorString(e));
  QE_CUDA(cudaSetDevice(cfg->device));
  DeviceInfo* d = nullptr;
  int32_t st = device_info(cfg->device, &d);
  if (st != QE_OK) return st;
  qe_ctx* c = new (std::nothrow) qe_ctx();
  if (!c) return fail(QE_ERR_BAD_ARG, "out of host memory");
  c->dev = d;
  c->exec_mode = cfg->exec_mode;
  c->one_way = (cfg->flags & QE_CTX_UNSAFE_ONE_WAY_HANDOFF) != 0;
  if (cfg->step_window) c->step_window = cfg->step_window > 64 ? 64 : cfg->step_window;
  e = cudaSuccess;
  if (cfg->exec_stream) {
    c->exec_stream = (cudaStream_t)cfg->exec_stream;
    c->owns_stream = false;
  } else {
    e = cudaStreamCreateWithFlags(&c->exec_stream, cudaStreamNonBlocking);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_in, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_out, cudaEventDisableTiming);
  if (e == cudaSuccess && (cfg->flags & QE_CTX_OVERLAP_DW)) {
    int least = 0, greatest = 0;
    e = cudaDeviceGetStreamPriorityRange(&least, &greatest);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&c->dw_stream, cudaStreamNonBlocking, least);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_dw_in, cudaEventDisableTiming);
  }
  st = e == cudaSuccess ? qe_registry_create(&c->registry) : fail(QE_ERR_CUDA, "context resources: %s", cudaGetErrorString(e));
  if (st != QE_OK) {  // release whatever was created
    if (c->ev_in) cudaEventDestroy(c->ev_in);
    if (c->ev_out) cudaEventDestroy(c->ev_out);
    if (c->ev_dw_in) cudaEventDestroy(c->ev_dw_in);
    if (c->dw_stream) cudaStreamDestroy(c->dw_stream);
    if (c->owns_stream && c->exec_stream) cudaStreamDestroy(c->exec_stream);
    delete c;
    return st;
  }
  *out = c;
  return QE_OK;
}

int32_t qe_ctx_destroy(qe_ctx* c) {
  if (!c || c->closed) return QE_OK;
  c->closed = true;
  ctx_release(c);
  return QE_OK;
}

int32_t qe_layer_workspace_bytes(const qe_layer_config* cfg, uint64_t* bytes_out) {
  int32_t st = check_config(cfg);
  if (st != QE_OK) return st;
  if (!bytes_out) return fail(QE_ERR_BAD_ARG, "bytes_out is null");
  *bytes_out = carve(*cfg).total;
  return QE_OK;
}

int32_t qe_layer_create(qe_ctx* ctx, const qe_layer_config* cfg, void* ws, uint64_t ws_bytes, qe_layer** out) {
  if (!ctx || !out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (ctx->closed) return fail(QE_ERR_BAD_ARG, "context already destroyed");
  int32_t st = check_config(cfg);
  if (st != QE_OK) return st;
  if (!cfg->weight_dev) return fail(QE_ERR_BAD_ARG, "weight_dev is null");
  const Carve k = carve(*cfg);
  if (!ws || ((uintptr_t)ws & 255u) || ws_bytes < k.total)
    return fail(QE_ERR_WORKSPACE, "workspace %p of %llu bytes; need %llu bytes, 256-byte aligned", ws,
                (unsigned long long)ws_bytes, (unsigned long long)k.total);
  qe_layer* L = new (std::nothrow) qe_layer();
  if (!L) return fail(QE_ERR_BAD_ARG, "out of host memory");
  L->ctx = ctx;
  L->cfg = *cfg;
  L->ws_bytes = k.total;
  st = qe_contract_create(cfg->slots, cfg->stage, cfg->unit, cfg->inv, ctx->registry, &L->contract);
  if (st != QE_OK) { delete L; return st; }
  uint8_t* base = (uint8_t*)ws;
  L->st = (qe::DevState*)base;
  L->hist = (float*)(base + k.hist);
  const bool wT = !qe::gemm_uses_pair(cfg->T), xgT = !qe::gemm_uses_pair(cfg->N);
  L->Wq = base + k.Wq;
  L->WqT = wT ? base + k.WqT : nullptr;
  if (cfg->host_io) {
    L->x_stage = base + k.stage_tk;
    L->dx_stage = L->x_stage + align_up(2ull * cfg->T * cfg->K, 1024);
    L->y_stage = base + k.stage_tn;
    L->dy_stage = L->y_stage + align_up(2ull * cfg->T * cfg->N, 1024);
  }
  const DeviceInfo* d = ctx->dev;
  const uint32_t T = cfg->T, K = cfg->K, N = cfg->N;
  for (uint32_t p = 0; p < cfg->slots; ++p) {
    uint8_t* s = base + k.slot0 + k.per_slot * p;
    L->Xq[p] = s + k.xq;
    L->XqT[p] = xgT ? s + k.xqT : nullptr;
    L->Gq[p] = s + k.gq;
    L->GqT[p] = xgT ? s + k.gqT : nullptr;
    if ((st = make_map(d, &L->tmXq_A[p], L->Xq[p], T, K, 128)) != QE_OK) break;   // F:  A = Xq  [T,K]
    if ((st = make_map(d, &L->tmGq_A[p], L->Gq[p], T, N, 128)) != QE_OK) break;   // dI: A = Gq  [T,N]
    if (xgT) {
      if ((st = make_map(d, &L->tmGqT_A[p], L->GqT[p], N, T, 128)) != QE_OK) break; // dW: A = Gq^T [N,T]
      if ((st = make_map(d, &L->tmXqT_B[p], L->XqT[p], K, T, qe::gemm_b_box_rows(N))) != QE_OK) break; // dW: B = Xq^T [K,T]
    } else {  // dW reads Gq [T,N] and Xq [T,K] as MN-major operands: 128 x 128 boxes over the row-major tensors
      if ((st = make_map(d, &L->tmGqT_A[p], L->Gq[p], T, N, 128)) != QE_OK) break;
      if ((st = make_map(d, &L->tmXqT_B[p], L->Xq[p], T, K, 128)) != QE_OK) break;
    }
  }
  if (st == QE_OK) st = make_map(d, &L->tmWq_B, L->Wq, N, K, qe::gemm_b_box_rows(T));    // F:  B = Wq   [N,K]
  if (st == QE_OK)  // dI: B = Wq^T [K,N], or Wq [N,K] itself as an MN-major operand
    st = wT ? make_map(d, &L->tmWqT_B, L->WqT, K, N, qe::gemm_b_box_rows(T)) : make_map(d, &L->tmWq_B_mn, L->Wq, N, K, 128);
  if (st != QE_OK) { qe_contract_destroy(L->contract); delete L; return st; }
  // state: histories 0, scales 1, everything else 0
  qe::DevState init{};
  for (int c = 0; c < 4; ++c) init.scale[c] = init.scale_inv[c] = 1.0f;
  cudaError_t e = cudaMemsetAsync(base, 0, k.Wq, ctx->exec_stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(base, &init, sizeof(init), cudaMemcpyHostToDevice, ctx->exec_stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->exec_stream);
  if (e != cudaSuccess) {
    qe_contract_destroy(L->contract);
    delete L;
    return fail(QE_ERR_CUDA, "state initialisation: %s", cudaGetErrorString(e));
  }
  if (ctx->dw_stream)
    for (uint32_t p = 0; p < cfg->slots; ++p) {
      cudaEventCreateWithFlags(&L->ev_di[p], cudaEventDisableTiming);
      cudaEventCreateWithFlags(&L->ev_dw[p], cudaEventDisableTiming);
    }
  ctx->stats.workspace_bytes += k.total;
  ctx->layers += 1;
  *out = L;
  return QE_OK;
}

int32_t qe_layer_destroy(qe_layer* L) {
  if (!L) return QE_OK;
  cudaStreamSynchronize(L->ctx->exec_stream);
  if (L->ctx->dw_stream) cudaStreamSynchronize(L->ctx->dw_stream);
  for (uint32_t p = 0; p < L->cfg.slots; ++p) {
    if (L->ev_di[p]) cudaEventDestroy(L->ev_di[p]);
    if (L->ev_dw[p]) cudaEventDestroy(L->ev_dw[p]);
    destroy_graph(&L->gF[p]);
    destroy_graph(&L->gDI[p]);
    destroy_graph(&L->gDW[p]);
    destroy_graph(&L->gDWs[p]);
  }
  destroy_graph(&L->gRefresh);
  destroy_graph(&L->gCommit);
  qe_ctx* ctx = L->ctx;
  ctx->stats.workspace_bytes -= L->ws_bytes;
  qe_contract_destroy(L->contract);
  delete L;
  ctx->layers -= 1;
  ctx_release(ctx);
  return QE_OK;
}

// x_host / y_host: non-null for the host-buffer entry point (x and y are then the layer's staging buffers)
static int32_t forward_impl(qe_layer* L, uint32_t mb, uint64_t gen, const void* x, void* y, void* caller_stream,
                            qe_tape* tape_out, const void* x_host, void* y_host) {
  int32_t refresh = 0;
  uint32_t p = 0;
  int32_t st = qe_contract_forward_check(L->contract, mb, gen, &refresh, &p);  // check ...
  if (st != QE_OK) return st;
  qe_ctx* ctx = L->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  const uint32_t T = L->cfg.T, K = L->cfg.K, N = L->cfg.N;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  if (x_host && (st = host_upload(ctx, const_cast<void*>(x), x_host, 2ull * T * K, caller)) != QE_OK) return st;
  if (L->dw_pending[p]) {  // the slot's buffers are still being read by the dW that released it (other stream)
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, L->ev_dw[p], 0));
    L->dw_pending[p] = false;
  }
  if (refresh) {
    std::vector<qe::Launch> rs;
    add_refresh(L, rs);
    if ((st = run_action(ctx, &L->gRefresh, rs)) != QE_OK) return st;
  }
  std::vector<qe::Launch> ls;
  add_forward(L, p, x, y, ls);
  if ((st = run_action(ctx, &L->gF[p], ls)) != QE_OK) return st;  // ... run ...
  if (x_host && (st = host_download(ctx, y_host, y, 2ull * T * N)) != QE_OK) return st;
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  return qe_contract_forward_commit(L->contract, mb, tape_out);  // ... commit
}

int32_t qe_forward(qe_layer* L, uint32_t mb, uint64_t gen, const void* x, void* y, void* caller_stream,
                   qe_tape* tape_out) {
  if (!L || !x || !y || !tape_out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (((uintptr_t)x | (uintptr_t)y) & 15u) return fail(QE_ERR_BAD_ARG, "x and y must be 16-byte aligned");
  return forward_impl(L, mb, gen, x, y, caller_stream, tape_out, nullptr, nullptr);
}

int32_t qe_forward_host(qe_layer* L, uint32_t mb, uint64_t gen, const void* x_host, void* y_host, void* caller_stream,
                        qe_tape* tape_out) {
  if (!L || !x_host || !tape_out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (!L->x_stage) return fail(QE_ERR_BAD_ARG, "layer was created without host_io");
  return forward_impl(L, mb, gen, L->x_stage, L->y_stage, caller_stream, tape_out, x_host, y_host);
}

static int32_t backward_dI_impl(qe_layer* L, const qe_tape* tape, const void* dy, void* dx, void* caller_stream,
                                const void* dy_host, void* dx_host) {
  int32_t st = qe_contract_dI_check(L->contract, tape);
  if (st != QE_OK) return st;
  qe_ctx* ctx = L->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  const uint32_t p = tape->ref.slot, T = L->cfg.T, K = L->cfg.K, N = L->cfg.N;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  if (dy_host && (st = host_upload(ctx, const_cast<void*>(dy), dy_host, 2ull * T * N, caller)) != QE_OK) return st;
  std::vector<qe::Launch> ls;
  add_dI(L, p, dy, dx, ls);
  if ((st = run_action(ctx, &L->gDI[p], ls)) != QE_OK) return st;
  if (ctx->dw_stream) QE_CUDA(cudaEventRecord(L->ev_di[p], ctx->exec_stream));
  if (dy_host && (st = host_download(ctx, dx_host, dx, 2ull * T * K)) != QE_OK) return st;
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  return qe_contract_dI_commit(L->contract, tape);
}

int32_t qe_backward_dI(qe_layer* L, const qe_tape* tape, const void* dy, void* dx, void* caller_stream) {
  if (!L || !tape || !dy || !dx) return fail(QE_ERR_BAD_ARG, "null argument");
  if (((uintptr_t)dy | (uintptr_t)dx) & 15u) return fail(QE_ERR_BAD_ARG, "dy and dx must be 16-byte aligned");
  return backward_dI_impl(L, tape, dy, dx, caller_stream, nullptr, nullptr);
}

int32_t qe_backward_dI_host(qe_layer* L, const qe_tape* tape, const void* dy_host, void* dx_host, void* caller_stream) {
  if (!L || !tape || !dy_host) return fail(QE_ERR_BAD_ARG, "null argument");
  if (!L->dy_stage) return fail(QE_ERR_BAD_ARG, "layer was created without host_io");
  return backward_dI_impl(L, tape, L->dy_stage, L->dx_stage, caller_stream, dy_host, dx_host);
}

// view != null: per-microbatch arena mode; grad / elems / off / slice then describe the layer's whole region of the
// arena in 4-byte units (what the contract core's destination rules are written in) and view is this microbatch's.
static int32_t backward_dW_impl(qe_layer* L, const qe_tape* tape, float* grad, uint64_t elems, uint64_t off,
                                float* temp, void* caller_stream, void* view = nullptr, uint64_t region_units = 0) {
  if (!L || !tape) return fail(QE_ERR_BAD_ARG, "null argument");
  const uint32_t K = L->cfg.K, N = L->cfg.N;
  const uint64_t slice = view ? region_units : (uint64_t)N * K;
  int32_t acc = 0;
  int32_t st = qe_contract_dW_check(L->contract, tape, (uint64_t)(uintptr_t)grad, elems, off, slice, &acc);
  if (st != QE_OK) return st;
  qe_ctx* ctx = L->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  const uint32_t p = tape->ref.slot;
  cudaStream_t run_on = ctx->exec_stream;
  if (ctx->dw_stream) {
    // overlapped dW: second stream, after the caller's work so far and after this tape's dI
    run_on = ctx->dw_stream;
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, caller));
    QE_CUDA(cudaStreamWaitEvent(run_on, ctx->ev_dw_in, 0));
    QE_CUDA(cudaStreamWaitEvent(run_on, L->ev_di[p], 0));
    ctx->stats.handoffs += 1;
  } else if ((st = handoff_in(ctx, caller)) != QE_OK) {
    return st;
  }
  std::vector<qe::Launch> ls;
  if (view) ls.push_back(qe::make_gemm(dW_gemm_view(L, p, view), ctx->dev->num_sms));
  else add_dW(L, p, grad + off, acc, temp, ls);
  st = run_action(ctx, temp ? &L->gDWs[p] : &L->gDW[p], ls, run_on);
  if (st != QE_OK) return st;
  if (ctx->dw_stream) {  // joined at the optimizer boundary and before the slot's next forward
    QE_CUDA(cudaEventRecord(L->ev_dw[p], run_on));
    L->dw_pending[p] = true;
  } else if ((st = handoff_out(ctx, caller)) != QE_OK) {
    return st;
  }
  return qe_contract_dW_commit(L->contract, tape, (uint64_t)(uintptr_t)grad, off, slice);
}

int32_t qe_backward_dW(qe_layer* L, const qe_tape* tape, float* grad, uint64_t elems, uint64_t off, void* stream) {
  return backward_dW_impl(L, tape, grad, elems, off, nullptr, stream);
}

int32_t qe_backward_dW_staged(qe_layer* L, const qe_tape* tape, float* grad, uint64_t elems, uint64_t off,
                              float* temp, void* stream) {
  if (!temp || ((uintptr_t)temp & 15u)) return fail(QE_ERR_BAD_ARG, "temp_dev must be non-null and 16-byte aligned");
  return backward_dW_impl(L, tape, grad, elems, off, temp, stream);
}

int32_t qe_backward_dW_arena(qe_layer* L, const qe_tape* tape, void* arena, uint64_t arena_elems, uint64_t layer_offset,
                             uint32_t microbatches, void* stream) {
  if (!L || !tape || !arena) return fail(QE_ERR_BAD_ARG, "null argument");
  if (microbatches < 1 || microbatches > QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "microbatches %u", microbatches);
  const uint64_t n = (uint64_t)L->cfg.N * L->cfg.K;
  if (layer_offset % 8 || ((uintptr_t)arena & 15u)) return fail(QE_ERR_DEST, "arena region not 16-byte aligned");
  if (tape->key.mb >= microbatches) return fail(QE_ERR_DEST, "microbatch %u has no view among %u", tape->key.mb, microbatches);
  uint16_t* view = (uint16_t*)arena + layer_offset + (uint64_t)tape->key.mb * n;
  // 2-byte elements expressed in the contract core's 4-byte units (n is even: N and K are multiples of 128)
  return backward_dW_impl(L, tape, (float*)arena, arena_elems / 2, layer_offset / 2, nullptr, stream, view, microbatches * n / 2);
}

int32_t qe_arena_finalize(qe_layer* L, const void* arena, uint64_t arena_elems, uint64_t layer_offset, uint32_t microbatches,
                          float* grad, uint64_t grad_elems, uint64_t off, void* caller_stream) {
  if (!L || !arena || !grad) return fail(QE_ERR_BAD_ARG, "null argument");
  if (microbatches < 1 || microbatches > QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "microbatches %u", microbatches);
  const qe_contract* c = L->contract;
  const uint64_t n = (uint64_t)L->cfg.N * L->cfg.K;
  if (c->aborted) return fail(QE_ERR_ABORTED, "step aborted; arena unusable for this epoch");
  const uint64_t want = microbatches == 64 ? ~0ull : ((1ull << microbatches) - 1);
  if (c->write_mask != want)
    return fail(QE_ERR_INCOMPLETE, "view write mask %#llx, expected %#llx", (unsigned long long)c->write_mask, (unsigned long long)want);
  if (!c->has_dest || c->dest_addr != (uint64_t)(uintptr_t)arena || c->dest_off != layer_offset / 2 || layer_offset % 8)
    return fail(QE_ERR_DEST, "not the arena region bound for this epoch");
  if (layer_offset > arena_elems || microbatches * n > arena_elems - layer_offset) return fail(QE_ERR_DEST, "region exceeds the arena");
  if (off > grad_elems || n > grad_elems - off || ((uintptr_t)(grad + off) & 15u)) return fail(QE_ERR_DEST, "gradient slice out of range or misaligned");
  qe_ctx* ctx = L->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  int32_t st = handoff_in(ctx, caller);
  if (st != QE_OK) return st;
  if (ctx->dw_stream) {  // the views were written on the second stream
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, ctx->dw_stream));
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_dw_in, 0));
  }
  qe::ArenaReduceParams ap{};
  ap.views = (const uint4*)((const uint16_t*)arena + layer_offset);
  ap.dst = (float4*)(grad + off);
  ap.view_vec = n / 8;
  ap.M = microbatches;
  if ((st = launch_eager(ctx, qe::make_arena_reduce(ap), ctx->exec_stream)) != QE_OK) return st;
  return handoff_out(ctx, caller);
}

static int32_t read_status(qe_layer* L, uint32_t* status) {
  QE_CUDA(cudaStreamSynchronize(L->ctx->exec_stream));
  if (L->ctx->dw_stream) QE_CUDA(cudaStreamSynchronize(L->ctx->dw_stream));
  QE_CUDA(cudaMemcpy(status, &L->st->status, sizeof(uint32_t), cudaMemcpyDeviceToHost));
  return QE_OK;
}

int32_t qe_optimizer_boundary(qe_layer* L, uint32_t expected) {
  if (!L) return fail(QE_ERR_BAD_ARG, "layer is null");
  uint32_t status = 0;
  int32_t st = read_status(L, &status);
  if (st != QE_OK) return st;
  if (status) return fail(QE_ERR_TIMEOUT, "device status word %#x: a bounded wait expired in a GEMM", status);
  return qe_contract_boundary(L->contract, expected);
}

int32_t qe_optimizer_boundary_all(qe_layer* const* layers, uint32_t n, uint32_t expected) {
  if (!layers || n < 1 || n > 4096) return fail(QE_ERR_BAD_ARG, "layers null or n = %u out of range", n);
  for (uint32_t i = 0; i < n; ++i) {
    if (!layers[i]) return fail(QE_ERR_BAD_ARG, "layers[%u] is null", i);
    if (layers[i]->ctx != layers[0]->ctx) return fail(QE_ERR_BAD_ARG, "layers[%u] belongs to another context", i);
  }
  qe_ctx* ctx = layers[0]->ctx;
  if (ctx->dw_stream) {  // deferred weight gradients run there: the gather below must come after them
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, ctx->dw_stream));
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_dw_in, 0));
  }
  uint32_t* out = &layers[0]->st->status_all;
  for (uint32_t lo = 0; lo < n; lo += 64) {
    qe::StatusGatherParams gp{};
    gp.n = std::min(64u, n - lo);
    for (uint32_t i = 0; i < gp.n; ++i) gp.src[i] = &layers[lo + i]->st->status;
    gp.out = out;
    gp.accumulate = lo ? 1u : 0u;
    QE_CUDA(launch_pdl(qe::make_status_gather(gp), ctx->exec_stream));
    ctx->stats.kernels_launched += 1;
  }
  uint32_t status = 0;
  QE_CUDA(cudaMemcpyAsync(&status, out, sizeof(status), cudaMemcpyDeviceToHost, ctx->exec_stream));
  QE_CUDA(cudaStreamSynchronize(ctx->exec_stream));  // the one drain: everything issued before the boundary is done
  if (status) return fail(QE_ERR_TIMEOUT, "device status word %#x: a bounded wait expired in a GEMM", status);
  for (uint32_t i = 0; i < n; ++i) {
    const int32_t st = qe_contract_boundary_check(layers[i]->contract, expected);
    if (st != QE_OK) return st;
  }
  for (uint32_t i = 0; i < n; ++i) qe_contract_boundary(layers[i]->contract, expected);
  return QE_OK;
}

int32_t qe_scale_commit(qe_layer* L, uint32_t cls, const float* amax_dev, void* caller_stream) {
  if (!L) return fail(QE_ERR_BAD_ARG, "layer is null");
  if (cls > QE_CLASS_Y) return fail(QE_ERR_BAD_ARG, "tensor_class %u", cls);
  qe_ctx* ctx = L->ctx;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  int32_t st;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  std::vector<qe::Launch> ls;
  ls.push_back(qe::make_commit(commit_params(L, 1u << cls, 0, amax_dev)));
  if ((st = run_action(ctx, &L->gCommit, ls)) != QE_OK) return st;
  return handoff_out(ctx, caller);
}

int32_t qe_abort_step(qe_layer* L) {
  if (!L) return fail(QE_ERR_BAD_ARG, "layer is null");
  return qe_contract_abort(L->contract);
}
int32_t qe_arena_rebuild(qe_layer* L) {
  if (!L) return fail(QE_ERR_BAD_ARG, "layer is null");
  return qe_contract_rebuild(L->contract);
}
int32_t qe_invalidate_cache(qe_layer* L) {
  if (!L) return fail(QE_ERR_BAD_ARG, "layer is null");
  return qe_contract_invalidate_cache(L->contract);
}
int32_t qe_next_slot(const qe_layer* L, uint32_t* slot_out) {
  if (!L || !slot_out) return fail(QE_ERR_BAD_ARG, "null argument");
  const int p = L->contract->lowest_free();
  if (p < 0) return fail(QE_ERR_POOL_FULL, "all slots occupied");
  *slot_out = (uint32_t)p;
  return QE_OK;
}

int32_t qe_get_state(qe_layer* L, qe_state_view* out, float* window_out, float* slot_sinv_out) {
  if (!L || !out) return fail(QE_ERR_BAD_ARG, "null argument");
  QE_CUDA(cudaStreamSynchronize(L->ctx->exec_stream));
  if (L->ctx->dw_stream) QE_CUDA(cudaStreamSynchronize(L->ctx->dw_stream));
  qe::DevState h;
  QE_CUDA(cudaMemcpy(&h, L->st, sizeof(h), cudaMemcpyDeviceToHost));
  std::memset(out, 0, sizeof(*out));
  for (int c = 0; c < 4; ++c) {
    out->cls[c].scale = h.scale[c];
    out->cls[c].scale_inv = h.scale_inv[c];
    out->cls[c].count = h.count[c];
  }
  out->cache_sinv_W = h.cache_sinv_W;
  out->device_status = h.status;
  out->device_token = h.token;
  int32_t st = qe_contract_get(L->contract, &out->contract);
  if (st != QE_OK) return st;
  const uint32_t H = L->cfg.history_len, P = L->cfg.slots;
  if (window_out) {
    std::vector<float> ring(4ull * H);
    QE_CUDA(cudaMemcpy(ring.data(), L->hist, ring.size() * sizeof(float), cudaMemcpyDeviceToHost));
    for (int c = 0; c < 4; ++c)
      for (uint32_t j = 0; j < H; ++j) {
        const uint64_t idx = ((uint64_t)h.count[c] + (uint64_t)H * 2 - 1 - j) % H;  // newest first
        window_out[(size_t)c * H + j] = ring[(size_t)c * H + idx];
      }
  }
  if (slot_sinv_out)
    for (uint32_t p = 0; p < P; ++p) {
      slot_sinv_out[p] = h.slot_sinv_X[p];
      slot_sinv_out[P + p] = h.slot_sinv_G[p];
    }
  return QE_OK;
}

int32_t qe_read_fp8(qe_layer* L, uint32_t which, uint32_t slot, void* host_out, uint64_t bytes) {
  if (!L || !host_out) return fail(QE_ERR_BAD_ARG, "null argument");
  const uint64_t tk = (uint64_t)L->cfg.T * L->cfg.K, tn = (uint64_t)L->cfg.T * L->cfg.N, nk = (uint64_t)L->cfg.N * L->cfg.K;
  if (which > 5 || (which < 4 && slot >= L->cfg.slots)) return fail(QE_ERR_BAD_ARG, "which %u slot %u", which, slot);
  const uint8_t* src = which == 0 ? L->Xq[slot] : which == 1 ? L->XqT[slot] : which == 2 ? L->Gq[slot]
                     : which == 3 ? L->GqT[slot] : which == 4 ? L->Wq : L->WqT;
  if (!src) return fail(QE_ERR_UNSUPPORTED, "this layer keeps no transposed copy %u (its GEMM reads the row-major tensor directly)", which);
  const uint64_t need = which < 2 ? tk : which < 4 ? tn : nk;
  if (bytes != need) return fail(QE_ERR_BAD_ARG, "bytes %llu, tensor has %llu", (unsigned long long)bytes, (unsigned long long)need);
  QE_CUDA(cudaStreamSynchronize(L->ctx->exec_stream));
  QE_CUDA(cudaMemcpy(host_out, src, need, cudaMemcpyDeviceToHost));
  return QE_OK;
}

// ------------------------------------------------------------------------------------------------ checkpoint
namespace {
struct StateHeader {
  uint32_t magic, version, T, K, N, H;
  int32_t margin;
  uint32_t reserved;
  uint64_t e_W;
  float scale[4], scale_inv[4];
  uint32_t count[4];
};
constexpr uint32_t kStateMagic = 0x53454651u;  // "QFES"
uint64_t state_bytes(const qe_layer* L) { return sizeof(StateHeader) + 4ull * L->cfg.history_len * sizeof(float); }
int32_t sync_layer(qe_layer* L) {
  QE_CUDA(cudaStreamSynchronize(L->ctx->exec_stream));
  if (L->ctx->dw_stream) QE_CUDA(cudaStreamSynchronize(L->ctx->dw_stream));
  return QE_OK;
}
}  // namespace

int32_t qe_state_bytes(const qe_layer* L, uint64_t* bytes_out) {
  if (!L || !bytes_out) return fail(QE_ERR_BAD_ARG, "null argument");
  *bytes_out = state_bytes(L);
  return QE_OK;
}

int32_t qe_state_save(qe_layer* L, void* host_out, uint64_t bytes) {
  if (!L || !host_out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (bytes != state_bytes(L)) return fail(QE_ERR_BAD_ARG, "bytes %llu, state has %llu", (unsigned long long)bytes, (unsigned long long)state_bytes(L));
  int32_t st = sync_layer(L);
  if (st != QE_OK) return st;
  if ((st = qe_contract_checkpoint_check(L->contract)) != QE_OK) return st;  // Invariant 4: only at quiescence
  qe::DevState h;
  QE_CUDA(cudaMemcpy(&h, L->st, sizeof(h), cudaMemcpyDeviceToHost));
  if (h.status) return fail(QE_ERR_TIMEOUT, "device status word %#x", h.status);
  StateHeader hd{};
  hd.magic = kStateMagic;
  hd.version = 1;
  hd.T = L->cfg.T;
  hd.K = L->cfg.K;
  hd.N = L->cfg.N;
  hd.H = L->cfg.history_len;
  hd.margin = L->cfg.margin;
  hd.e_W = L->contract->e_W;
  for (int c = 0; c < 4; ++c) {
    hd.scale[c] = h.scale[c];
    hd.scale_inv[c] = h.scale_inv[c];
    hd.count[c] = h.count[c];
  }
  std::memcpy(host_out, &hd, sizeof(hd));
  QE_CUDA(cudaMemcpy((char*)host_out + sizeof(hd), L->hist, 4ull * hd.H * sizeof(float), cudaMemcpyDeviceToHost));
  return QE_OK;
}

int32_t qe_state_load(qe_layer* L, const void* host_in, uint64_t bytes) {
  if (!L || !host_in) return fail(QE_ERR_BAD_ARG, "null argument");
  if (bytes != state_bytes(L)) return fail(QE_ERR_BAD_ARG, "bytes %llu, state has %llu", (unsigned long long)bytes, (unsigned long long)state_bytes(L));
  StateHeader hd;
  std::memcpy(&hd, host_in, sizeof(hd));
  if (hd.magic != kStateMagic || hd.version != 1) return fail(QE_ERR_BAD_ARG, "not a layer state payload");
  if (hd.T != L->cfg.T || hd.K != L->cfg.K || hd.N != L->cfg.N || hd.H != L->cfg.history_len || hd.margin != L->cfg.margin)
    return fail(QE_ERR_SHAPE, "payload is for T=%u K=%u N=%u H=%u margin=%d", hd.T, hd.K, hd.N, hd.H, hd.margin);
  int32_t st = sync_layer(L);
  if (st != QE_OK) return st;
  if ((st = qe_contract_restore(L->contract, hd.e_W)) != QE_OK) return st;  // fails, changing nothing, if a tape lives
  qe::DevState h;
  QE_CUDA(cudaMemcpy(&h, L->st, sizeof(h), cudaMemcpyDeviceToHost));
  for (int c = 0; c < 4; ++c) {
    h.scale[c] = hd.scale[c];
    h.scale_inv[c] = hd.scale_inv[c];
    h.count[c] = hd.count[c];
    h.pending_amax[c] = 0;
    // derived state: the maximum of the restored ring (bit patterns of non-negative values order like the values)
    const uint32_t* ring = reinterpret_cast<const uint32_t*>((const char*)host_in + sizeof(hd)) + (size_t)c * hd.H;
    uint32_t m = 0;
    for (uint32_t i = 0; i < hd.H; ++i) m = ring[i] > m ? ring[i] : m;
    h.wmax[c] = m;
  }
  h.cache_sinv_W = 0.0f;  // cache contents are rebuilt by the first forward
  QE_CUDA(cudaMemcpy(L->st, &h, sizeof(h), cudaMemcpyHostToDevice));
  QE_CUDA(cudaMemcpy(L->hist, (const char*)host_in + sizeof(hd), 4ull * hd.H * sizeof(float), cudaMemcpyHostToDevice));
  return QE_OK;
}

int32_t qe_get_stats(const qe_ctx* ctx, qe_stats* out) {
  if (!ctx || !out) return fail(QE_ERR_BAD_ARG, "null argument");
  *out = ctx->stats;
  return QE_OK;
}

}  // extern "C"
