// Execution layer and launch builders of the layer API (definitions of layer_impl.h).
#include "layer_impl.h"

namespace qe_impl {

DeviceInfo g_dev[16];

// Per-device one-time setup: SM count, compute capability, driver entry point for tensor-map encoding, and the
// GEMM's shared-memory opt-in.  The device must be current.
int32_t device_info(int device, DeviceInfo** out) {
  if (device < 0 || device >= 16) return fail(QE_ERR_BAD_ARG, "device %d", device);
  DeviceInfo& d = g_dev[device];
  if (!d.ready) {
    cudaDeviceProp prop;
    QE_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return fail(QE_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library needs sm_100", device, prop.major, prop.minor);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    QE_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return fail(QE_ERR_CUDA, "cuTensorMapEncodeTiled not available");
    QE_CUDA(qe::gemm_prepare());
    d.device = device;
    d.num_sms = prop.multiProcessorCount;
    d.cc_major = prop.major;
    d.encode = (EncodeTiledFn)fn;
    d.ready = true;
  }
  *out = &d;
  return QE_OK;
}

// Tensor map over a contraction-major byte matrix [rows, inner]: box = 128 bytes x box_rows, 128-byte swizzle.
int32_t make_map(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t inner,
                 uint32_t box_rows) {
  cuuint64_t gdim[2] = {inner, rows};
  cuuint64_t gstride[1] = {inner};
  cuuint32_t box[2] = {128u, box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = d->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(QE_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
  return QE_OK;
}

// Tensor map over the output D [M, N] (row pitch ldo elements) for the epilogue's bulk stores: 32 x 32 boxes; bf16
// rows of a box are 64 bytes (64-byte swizzle), FP32 rows 128 bytes (128-byte swizzle).
int32_t make_out_map(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t M, uint64_t N, uint64_t ldo,
                     bool fp32) {
  cuuint64_t gdim[2] = {N, M};
  cuuint64_t gstride[1] = {ldo * (fp32 ? 4u : 2u)};
  cuuint32_t box[2] = {32u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = d->encode(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                         const_cast<void*>(ptr), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         fp32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(QE_ERR_CUDA, "cuTensorMapEncodeTiled (output) failed with %d", (int)r);
  return QE_OK;
}

// Tensor map over FP8 bytes D [M, N] (row pitch ld bytes) for the hand-off epilogue: 32-byte x 32-row boxes, no swizzle.
int32_t make_out_map_u8(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t M, uint64_t N, uint64_t ld) {
  cuuint64_t gdim[2] = {N, M};
  cuuint64_t gstride[1] = {ld};
  cuuint32_t box[2] = {32u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = d->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(QE_ERR_CUDA, "cuTensorMapEncodeTiled (FP8 output) failed with %d", (int)r);
  return QE_OK;
}


int32_t current_device_info(DeviceInfo** d) {
  int dev = 0;
  QE_CUDA(cudaGetDevice(&dev));
  return device_info(dev, d);
}

int32_t launch_on(const qe::Launch& l, cudaStream_t s) {
  QE_CUDA(launch_pdl(l, s));
  return QE_OK;
}


void destroy_graph(ActionGraph* g) {
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  g->exec = nullptr;
  g->graph = nullptr;
  g->built = false;
}
void ctx_release(qe_ctx* c) {
  if (!c->closed || c->layers) return;
  cudaStreamSynchronize(c->exec_stream);
  for (auto* sg : c->step_graphs) {
    destroy_graph(&sg->g);
    delete sg;
  }
  if (c->dw_stream) {
    cudaStreamSynchronize(c->dw_stream);
    cudaStreamDestroy(c->dw_stream);
    cudaEventDestroy(c->ev_dw_in);
  }
  if (c->h2d_stream) {
    cudaStreamSynchronize(c->h2d_stream);
    cudaStreamSynchronize(c->d2h_stream);
    cudaStreamDestroy(c->h2d_stream);
    cudaStreamDestroy(c->d2h_stream);
    cudaEventDestroy(c->ev_h2d);
    cudaEventDestroy(c->ev_kernels);
    cudaEventDestroy(c->ev_d2h);
  }
  cudaEventDestroy(c->ev_in);
  cudaEventDestroy(c->ev_out);
  if (c->owns_stream) cudaStreamDestroy(c->exec_stream);
  qe_registry_destroy(c->registry);
  delete c;
}



// One launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the stream
// drains; every kernel of the library waits for its predecessors (griddepcontrol.wait) before touching their data.
cudaError_t launch_pdl(const qe::Launch& l, cudaStream_t stream) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = l.grid;
  cfg.blockDim = l.block;
  cfg.dynamicSmemBytes = l.smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  void* args[1] = {const_cast<unsigned char*>(l.params)};
  return cudaLaunchKernelExC(&cfg, l.func, args);
}

int32_t launch_eager(qe_ctx* ctx, const qe::Launch& l, cudaStream_t stream) {
  QE_CUDA(launch_pdl(l, stream));
  ctx->stats.eager_launches += 1;
  ctx->stats.kernels_launched += 1;
  return QE_OK;
}

// Capture the launches on the execution stream into a graph, instantiate it, and recover the kernel nodes in
// launch order by walking the (linear) dependency chain from the root.
int32_t build_graph(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream) {
  const auto t0 = std::chrono::steady_clock::now();
  QE_CUDA(cudaStreamBeginCapture(stream, cudaStreamCaptureModeThreadLocal));
  cudaError_t err = cudaSuccess;
  for (const qe::Launch& l : ls) {
    err = launch_pdl(l, stream);
    if (err != cudaSuccess) break;
  }
  cudaGraph_t graph = nullptr;
  cudaError_t end = cudaStreamEndCapture(stream, &graph);
  if (err != cudaSuccess) {
    if (graph) cudaGraphDestroy(graph);
    return fail(QE_ERR_CUDA, "launch during capture: %s", cudaGetErrorString(err));
  }
  QE_CUDA(end);
  size_t n = 0;
  QE_CUDA(cudaGraphGetNodes(graph, nullptr, &n));
  if (n != ls.size()) {
    cudaGraphDestroy(graph);
    return fail(QE_ERR_CUDA, "captured %zu nodes for %zu launches", n, ls.size());
  }
  std::vector<cudaGraphNode_t> chain;
  size_t nroot = 1;
  cudaGraphNode_t cur = nullptr;
  QE_CUDA(cudaGraphGetRootNodes(graph, &cur, &nroot));
  if (nroot != 1) {
    cudaGraphDestroy(graph);
    return fail(QE_ERR_CUDA, "captured graph has %zu roots", nroot);
  }
  while (cur) {
    chain.push_back(cur);
    // the edges carry programmatic-dependency data, which only the _v2 query reports
    size_t nd = 0;
    QE_CUDA(cudaGraphNodeGetDependentNodes_v2(cur, nullptr, nullptr, &nd));
    if (nd == 0) break;
    if (nd != 1) return fail(QE_ERR_CUDA, "captured graph is not a chain");
    cudaGraphNode_t next = nullptr;
    cudaGraphEdgeData edge{};
    QE_CUDA(cudaGraphNodeGetDependentNodes_v2(cur, &next, &edge, &nd));
    cur = next;
  }
  if (chain.size() != ls.size()) {
    cudaGraphDestroy(graph);
    return fail(QE_ERR_CUDA, "chain of %zu nodes for %zu launches", chain.size(), ls.size());
  }
  cudaGraphExec_t exec = nullptr;
  cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
  if (ie != cudaSuccess) {
    cudaGraphDestroy(graph);
    return fail(QE_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(ie));
  }
  g->graph = graph;
  g->exec = exec;
  g->nodes = chain;
  g->launches = ls;
  g->built = true;
  ctx->stats.graphs_built += 1;
  ctx->stats.capture_host_ms += std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
  return QE_OK;
}

int32_t replay_graph(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream) {
  if (ls.size() != g->launches.size()) return fail(QE_ERR_CUDA, "graph shape changed");
  for (size_t i = 0; i < ls.size(); ++i) {
    const qe::Launch& now = ls[i];
    qe::Launch& was = g->launches[i];
    const bool same = now.func == was.func && now.nbytes == was.nbytes && now.smem == was.smem &&
                      now.grid.x == was.grid.x && now.grid.y == was.grid.y && now.block.x == was.block.x &&
                      std::memcmp(now.params, was.params, now.nbytes) == 0;
    if (same) continue;
    // caller-visible pointers (x, y, gradient destination) or the accumulate flag changed: patch the node in place
    cudaKernelNodeParams np{};
    void* args[1] = {const_cast<unsigned char*>(now.params)};
    np.func = const_cast<void*>(now.func);
    np.gridDim = now.grid;
    np.blockDim = now.block;
    np.sharedMemBytes = now.smem;
    np.kernelParams = args;
    np.extra = nullptr;
    QE_CUDA(cudaGraphExecKernelNodeSetParams(g->exec, g->nodes[i], &np));
    was = now;
    ctx->stats.node_param_updates += 1;
  }
  QE_CUDA(cudaGraphLaunch(g->exec, stream));
  ctx->stats.graph_replays += 1;
  ctx->stats.kernels_launched += ls.size();
  return QE_OK;
}

// Sec. 4.4: the execution stream waits on the caller's stream before the action...
int32_t handoff_in(qe_ctx* ctx, cudaStream_t caller) {
  if (caller == ctx->exec_stream) return QE_OK;
  QE_CUDA(cudaEventRecord(ctx->ev_in, caller));
  QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_in, 0));
  ctx->stats.handoffs += 1;
  return QE_OK;
}
// ...and the caller's stream waits on the action's tail before it may consume anything.
int32_t handoff_out(qe_ctx* ctx, cudaStream_t caller) {
  if (caller == ctx->exec_stream) return QE_OK;
  if (ctx->one_way) return QE_OK;  // the defective protocol, kept for the stale-read experiment only
  QE_CUDA(cudaEventRecord(ctx->ev_out, ctx->exec_stream));
  QE_CUDA(cudaStreamWaitEvent(caller, ctx->ev_out, 0));
  ctx->stats.handoffs += 1;
  return QE_OK;
}

// ---- host-buffer calls.  The upload of an action runs on one copy stream and the read-back of its result on
// another, so that the upload of action k+1 overlaps the read-back of action k (the host link is full duplex); the
// kernels stay on the execution stream, which waits for the upload before them and for the read-back after them
// (a caller that synchronises after the call finds its host buffer complete).
int32_t host_upload(qe_ctx* ctx, void* dst, const void* src_host, size_t bytes, cudaStream_t caller) {
  if (!ctx->h2d_stream) {
    cudaError_t e = cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_h2d, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_kernels, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_d2h, cudaEventDisableTiming);
    if (e != cudaSuccess) return fail(QE_ERR_CUDA, "copy streams: %s", cudaGetErrorString(e));
  }
  // the staging buffer was last read by the kernels of an earlier host-buffer call
  if (ctx->kernels_recorded) QE_CUDA(cudaStreamWaitEvent(ctx->h2d_stream, ctx->ev_kernels, 0));
  if (caller != ctx->exec_stream) QE_CUDA(cudaStreamWaitEvent(ctx->h2d_stream, ctx->ev_in, 0));  // recorded by handoff_in
  QE_CUDA(cudaMemcpyAsync(dst, src_host, bytes, cudaMemcpyHostToDevice, ctx->h2d_stream));
  QE_CUDA(cudaEventRecord(ctx->ev_h2d, ctx->h2d_stream));
  QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_h2d, 0));
  return QE_OK;
}
// after the action's kernels: frees the staging input for the next upload and starts the read-back (if any)
int32_t host_download(qe_ctx* ctx, void* dst_host, const void* src, size_t bytes) {
  QE_CUDA(cudaEventRecord(ctx->ev_kernels, ctx->exec_stream));
  ctx->kernels_recorded = true;
  if (!dst_host) return QE_OK;
  QE_CUDA(cudaStreamWaitEvent(ctx->d2h_stream, ctx->ev_kernels, 0));
  QE_CUDA(cudaMemcpyAsync(dst_host, src, bytes, cudaMemcpyDeviceToHost, ctx->d2h_stream));
  QE_CUDA(cudaEventRecord(ctx->ev_d2h, ctx->d2h_stream));
  QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_d2h, 0));
  return QE_OK;
}

int32_t run_action(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream) {
  if (!stream) stream = ctx->exec_stream;
  if (ctx->exec_mode == QE_EXEC_GRAPH) {
    if (!g->built) {
      int32_t st = build_graph(ctx, g, ls, stream);
      if (st != QE_OK) return st;
    }
    return replay_graph(ctx, g, ls, stream);
  }
  for (const qe::Launch& l : ls) {
    int32_t st = launch_eager(ctx, l, stream);
    if (st != QE_OK) return st;
  }
  return QE_OK;
}

// Graph of a launch list identified by a hash (whole steps, multi-layer dW calls); rebuilt when the list's length
// changed under the same key (e.g. no weight refresh this time).
ActionGraph* keyed_graph(qe_ctx* ctx, uint64_t key, size_t n_launches) {
  qe_ctx::StepGraph* sg = nullptr;
  for (auto* c : ctx->step_graphs)
    if (c->key == key) sg = c;
  if (sg && sg->g.launches.size() != n_launches) {
    destroy_graph(&sg->g);
    sg->g = ActionGraph();
  }
  if (!sg) {
    sg = new (std::nothrow) qe_ctx::StepGraph();
    if (!sg) return nullptr;
    sg->key = key;
    ctx->step_graphs.push_back(sg);
  }
  return &sg->g;
}


int32_t run_keyed(qe_ctx* ctx, uint64_t key, const std::vector<qe::Launch>& ls) {
  if (ctx->exec_mode == QE_EXEC_GRAPH) {
    ActionGraph* g = keyed_graph(ctx, key, ls.size());
    if (!g) return fail(QE_ERR_BAD_ARG, "out of host memory");
    return run_action(ctx, g, ls);
  }
  for (const qe::Launch& l : ls) {
    int32_t st = launch_eager(ctx, l, ctx->exec_stream);
    if (st != QE_OK) return st;
  }
  return QE_OK;
}




Carve carve(const qe_layer_config& c) {
  Carve k{};
  uint64_t o = sizeof(qe::DevState);
  k.hist = o;
  o = align_up(o + 4ull * c.history_len * sizeof(float), 1024);
  const uint64_t nk = (uint64_t)c.N * c.K, tk = (uint64_t)c.T * c.K, tn = (uint64_t)c.T * c.N;
  // Transposed FP8 copies exist only where a GEMM cannot take the row-major tensor as an MN-major operand: the dI
  // GEMM (M = T) needs Wq^T, the dW GEMM (M = N) needs Xq^T and Gq^T, when that M is not a multiple of 256.
  const bool wT = !qe::gemm_uses_pair(c.T), xgT = !qe::gemm_uses_pair(c.N);
  k.Wq = o;
  o += align_up(nk, 1024);
  k.WqT = o;
  if (wT) o += align_up(nk, 1024);
  k.slot0 = o;
  k.xq = 0;
  k.xqT = align_up(tk, 1024);
  k.gq = k.xqT + (xgT ? align_up(tk, 1024) : 0);
  k.gqT = k.gq + align_up(tn, 1024);
  k.per_slot = k.gqT + (xgT ? align_up(tn, 1024) : 0);
  o += k.per_slot * c.slots;
  if (c.host_io) {  // x / dx [T,K] and y / dy [T,N] bf16 staging for the host-buffer entry points
    k.stage_tk = o;
    o += 2 * align_up(2 * tk, 1024);
    k.stage_tn = o;
    o += 2 * align_up(2 * tn, 1024);
  }
  k.total = o;
  return k;
}

int32_t check_config(const qe_layer_config* c) {
  if (!c) return fail(QE_ERR_BAD_ARG, "config is null");
  if (!shape_ok(c->T) || !shape_ok(c->K) || !shape_ok(c->N))
    return fail(QE_ERR_SHAPE, "T=%u K=%u N=%u: each must be a multiple of 128 in [256, 2^20]", c->T, c->K, c->N);
  if (c->history_len < 1 || c->history_len > QE_MAX_HISTORY) return fail(QE_ERR_BAD_ARG, "history_len %u", c->history_len);
  if (c->margin < -32 || c->margin > 32) return fail(QE_ERR_BAD_ARG, "margin %d", c->margin);
  if (c->slots < 1 || c->slots > QE_MAX_SLOTS) return fail(QE_ERR_BAD_ARG, "slots %u", c->slots);
  if (c->host_io > 1) return fail(QE_ERR_BAD_ARG, "host_io %u", c->host_io);
  return QE_OK;
}

qe::CommitParams commit_params(qe_layer* L, uint32_t mask, uint32_t bump, const float* override_amax) {
  qe::CommitParams cp{};
  cp.st = L->st;
  cp.hist = L->hist;
  cp.H = L->cfg.history_len;
  cp.class_mask = mask;
  cp.pow2_neg_margin = std::ldexp(1.0f, -L->cfg.margin);
  cp.amax_override = override_amax;
  cp.bump_token = bump;
  return cp;
}

// commit_mask != 0: the kernel's last block also commits those classes (used for the weight refresh)
qe::QuantParams quant_params(qe_layer* L, const void* x, uint8_t* q, uint8_t* qT, uint32_t rows, uint32_t cols, int cls,
                             float* sinv_dst, int fmt, uint32_t commit_mask) {
  qe::QuantParams qp{};
  qp.x = (const uint16_t*)x;
  qp.q = q;
  qp.qT = qT;
  qp.rows = rows;
  qp.cols = cols;
  qp.scale = &L->st->scale[cls];
  qp.sinv_src = &L->st->scale_inv[cls];
  qp.sinv_dst = sinv_dst;
  qp.amax_bits = &L->st->pending_amax[cls];
  qp.fmt = fmt;
  if (commit_mask) qp.commit = commit_params(L, commit_mask, 0, nullptr);
  return qp;
}
qe::Launch quant_launch(qe_layer* L, const void* x, uint8_t* q, uint8_t* qT, uint32_t rows, uint32_t cols, int cls,
                        float* sinv_dst, int fmt, uint32_t commit_mask) {
  return qe::make_quantize(quant_params(L, x, q, qT, rows, cols, cls, sinv_dst, fmt, commit_mask));
}


// ---- the launches of each action (shared by the per-action calls and the whole-step call)
void add_refresh(qe_layer* L, std::vector<qe::Launch>& ls) {
  // Invariant 3: first forward of the epoch re-quantises the weight; the kernel's last block commits its amax
  ls.push_back(quant_launch(L, L->cfg.weight_dev, L->Wq, L->WqT, L->cfg.N, L->cfg.K, QE_CLASS_W, &L->st->cache_sinv_W,
                            QE_E4M3, 1u << QE_CLASS_W));
}

// FP8 hand-off between directly chained linears: the forward GEMM of `L` emits its output as the E4M3 input of
// `next` (quantised with next's current X scale, straight into next's tape slot pn, with next's X amax and
// inverse-scale snapshot), so `next` needs no cast kernel; x == null means L's own input was deposited that way.
// gemm_out != null: the GEMM is handed back instead of being queued (the caller puts it into a shared launch).
void add_forward(qe_layer* L, uint32_t p, const void* x, void* y, std::vector<qe::Launch>& ls, qe_layer* next,
                 uint32_t pn, qe::GemmParams* gemm_out, qe::QuantParams* cast_out) {
  const uint32_t T = L->cfg.T, K = L->cfg.K, N = L->cfg.N;
  if (x && cast_out) *cast_out = quant_params(L, x, L->Xq[p], L->XqT[p], T, K, QE_CLASS_X, &L->st->slot_sinv_X[p], QE_E4M3);
  else if (x) ls.push_back(quant_launch(L, x, L->Xq[p], L->XqT[p], T, K, QE_CLASS_X, &L->st->slot_sinv_X[p], QE_E4M3));
  qe::GemmParams gp{};
  gp.tmA = L->tmXq_A[p];
  gp.tmB = L->tmWq_B;
  gp.M = T;
  gp.N = N;
  gp.Kc = K;
  gp.idesc = qe::gemm_idesc(QE_E4M3, QE_E4M3, T);
  gp.alpha_a = &L->st->slot_sinv_X[p];
  gp.alpha_b = &L->st->cache_sinv_W;
  gp.ldo = N;
  if (next) {
    gp.out = next->Xq[pn];
    gp.epi = 3;
    make_out_map_u8(L->ctx->dev, &gp.tmD, next->Xq[pn], T, N, N);
    gp.out_scale = &next->st->scale[QE_CLASS_X];
    gp.out_fmt = QE_E4M3;
    gp.amax_bits2 = &next->st->pending_amax[QE_CLASS_X];
    gp.sinv_src = &next->st->scale_inv[QE_CLASS_X];
    gp.sinv_dst = &next->st->slot_sinv_X[pn];
  } else {
    gp.out = y;
    gp.epi = 0;
    make_out_map(L->ctx->dev, &gp.tmD, y, T, N, N, false);
  }
  gp.amax_bits = &L->st->pending_amax[QE_CLASS_Y];
  gp.status = &L->st->status;
  gp.commit = commit_params(L, (1u << QE_CLASS_X) | (1u << QE_CLASS_Y), 1, nullptr);  // done by the GEMM's last CTA
  if (gemm_out) *gemm_out = gp;
  else ls.push_back(qe::make_gemm(gp, L->ctx->dev->num_sms));
}

// Hand-off in the backward direction: the input gradient of `L` is the output gradient of the linear before it
// (`prev`), emitted as E5M2 with prev's G scale into prev's tape slot pp; dy == null: L's own dY came that way.
void add_dI(qe_layer* L, uint32_t p, const void* dy, void* dx, std::vector<qe::Launch>& ls, qe_layer* prev,
            uint32_t pp, qe::GemmParams* gemm_out, qe::QuantParams* cast_out) {
  const uint32_t T = L->cfg.T, K = L->cfg.K, N = L->cfg.N;
  if (dy && cast_out) *cast_out = quant_params(L, dy, L->Gq[p], L->GqT[p], T, N, QE_CLASS_G, &L->st->slot_sinv_G[p], QE_E5M2);
  else if (dy) ls.push_back(quant_launch(L, dy, L->Gq[p], L->GqT[p], T, N, QE_CLASS_G, &L->st->slot_sinv_G[p], QE_E5M2));
  qe::GemmParams gp{};
  const bool b_mn = L->WqT == nullptr;  // no transposed weight copy: Wq [N,K] is B in MN-major form
  gp.tmA = L->tmGq_A[p];
  gp.tmB = b_mn ? L->tmWq_B_mn : L->tmWqT_B;
  gp.M = T;
  gp.N = K;
  gp.Kc = N;
  gp.idesc = qe::gemm_idesc(QE_E5M2, QE_E4M3, T, false, b_mn);
  gp.b_mn = b_mn;
  gp.alpha_a = &L->st->slot_sinv_G[p];
  gp.alpha_b = &L->st->cache_sinv_W;
  gp.ldo = K;
  if (prev) {
    gp.out = prev->Gq[pp];
    gp.epi = 3;
    make_out_map_u8(L->ctx->dev, &gp.tmD, prev->Gq[pp], T, K, K);
    gp.out_scale = &prev->st->scale[QE_CLASS_G];
    gp.out_fmt = QE_E5M2;
    gp.amax_bits2 = &prev->st->pending_amax[QE_CLASS_G];
    gp.sinv_src = &prev->st->scale_inv[QE_CLASS_G];
    gp.sinv_dst = &prev->st->slot_sinv_G[pp];
  } else {
    gp.out = dx;
    gp.epi = 0;
    make_out_map(L->ctx->dev, &gp.tmD, dx, T, K, K, false);
  }
  gp.amax_bits = nullptr;
  gp.status = &L->st->status;
  gp.commit = commit_params(L, 1u << QE_CLASS_G, 1, nullptr);  // backward amax/scale updated exactly once, here
  if (gemm_out) *gemm_out = gp;
  else ls.push_back(qe::make_gemm(gp, L->ctx->dev->num_sms));
}

// The weight-gradient GEMM of slot p; dst = first element of the layer's gradient slice, temp != null makes it
// write the temporary instead (copied-gradient comparison path).
qe::GemmParams dW_gemm(qe_layer* L, uint32_t p, float* dst, int32_t accumulate, float* temp) {
  const uint32_t T = L->cfg.T, K = L->cfg.K, N = L->cfg.N;
  qe::GemmParams gp{};
  const bool mn = L->GqT[p] == nullptr;  // Gq [T,N] and Xq [T,K] themselves, read as MN-major operands
  gp.tmA = L->tmGqT_A[p];
  gp.tmB = L->tmXqT_B[p];
  gp.M = N;
  gp.N = K;
  gp.Kc = T;
  gp.idesc = qe::gemm_idesc(QE_E5M2, QE_E4M3, N, mn, mn);
  gp.a_mn = gp.b_mn = mn;
  gp.alpha_a = &L->st->slot_sinv_G[p];  // snapshots taken when dY_m and X_m were quantised, never the current state
  gp.alpha_b = &L->st->slot_sinv_X[p];
  gp.ldo = K;
  gp.amax_bits = nullptr;
  gp.status = &L->st->status;
  make_out_map(L->ctx->dev, &gp.tmD, temp ? temp : dst, N, K, K, true);  // used by the overwrite epilogue
  if (!temp) {
    gp.out = dst;  // direct placement: the epilogue reads, adds and writes the destination itself
    gp.epi = accumulate ? 2 : 1;
  } else {
    gp.out = temp;
    gp.epi = 1;
  }
  return gp;
}

// Per-microbatch arena: the same GEMM writes bf16(D) into the microbatch's own view (no accumulation, no amax).
qe::GemmParams dW_gemm_view(qe_layer* L, uint32_t p, void* view) {
  qe::GemmParams gp = dW_gemm(L, p, nullptr, 0, nullptr);
  gp.out = view;
  gp.epi = 0;
  make_out_map(L->ctx->dev, &gp.tmD, view, L->cfg.N, L->cfg.K, L->cfg.K, false);
  return gp;
}

void add_dW(qe_layer* L, uint32_t p, float* dst, int32_t accumulate, float* temp, std::vector<qe::Launch>& ls) {
  const uint32_t K = L->cfg.K, N = L->cfg.N;
  ls.push_back(qe::make_gemm(dW_gemm(L, p, dst, accumulate, temp), L->ctx->dev->num_sms));
  if (temp) {
    qe::AccumParams ap{};
    ap.dst = (float4*)dst;
    ap.src = (const float4*)temp;
    ap.nvec = (uint64_t)N * K / 4;
    ap.accumulate = accumulate;
    ls.push_back(qe::make_accumulate(ap));
  }
}


}  // namespace qe_impl
