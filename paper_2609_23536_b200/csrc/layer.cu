// Host side of the layer API: workspace carve-up, tensor maps, the three checked actions and the execution layer
// (eager launches or one CUDA graph per (action, slot), both bracketed by the two-way stream handshake).
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "contract.h"
#include "error.h"
#include "kernels.h"
#include "qe.h"

using qe::fail;

#define QE_CUDA(expr)                                                                         \
  do {                                                                                        \
    cudaError_t e_ = (expr);                                                                  \
    if (e_ != cudaSuccess) return fail(QE_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceInfo {
  bool ready = false;
  int device = -1, num_sms = 0, cc_major = 0;
  EncodeTiledFn encode = nullptr;
};
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

uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

bool shape_ok(uint32_t v) { return v >= 256 && v % 128 == 0 && v <= (1u << 20); }

}  // namespace

// ================================================================================================ execution layer
struct ActionGraph {
  bool built = false;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  std::vector<cudaGraphNode_t> nodes;
  std::vector<qe::Launch> launches;
};

struct qe_ctx {
  DeviceInfo* dev = nullptr;
  uint32_t exec_mode = QE_EXEC_EAGER;
  cudaStream_t exec_stream = nullptr;
  bool owns_stream = true;
  bool one_way = false;              // QE_CTX_UNSAFE_ONE_WAY_HANDOFF
  uint32_t step_window = 4;          // qe_step_run: units looked ahead when planning rounds (1: action by action)
  cudaStream_t dw_stream = nullptr;  // only with QE_CTX_OVERLAP_DW
  cudaEvent_t ev_dw_in = nullptr;
  cudaEvent_t ev_in = nullptr, ev_out = nullptr;
  // host-buffer calls: copy streams and their events, created by the first such call
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_h2d = nullptr, ev_kernels = nullptr, ev_d2h = nullptr;
  bool kernels_recorded = false;
  qe_registry* registry = nullptr;
  qe_stats stats{};
  // Layers keep their context alive: it is released when the caller has destroyed it AND its last layer is gone,
  // so the two destroy calls may come in either order.
  uint32_t layers = 0;
  bool closed = false;
  // whole-step graphs, one per distinct (layers, actions) list
  struct StepGraph { uint64_t key; ActionGraph g; };
  std::vector<StepGraph*> step_graphs;
};

static void destroy_graph(ActionGraph* g);

static void ctx_release(qe_ctx* c) {
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

struct qe_layer {
  qe_ctx* ctx = nullptr;
  qe_layer_config cfg{};
  qe_contract* contract = nullptr;
  uint64_t ws_bytes = 0;
  qe::DevState* st = nullptr;
  float* hist = nullptr;
  uint8_t *Wq = nullptr, *WqT = nullptr;
  uint8_t *x_stage = nullptr, *dx_stage = nullptr, *y_stage = nullptr, *dy_stage = nullptr;  // host_io only
  uint8_t *Xq[QE_MAX_SLOTS], *XqT[QE_MAX_SLOTS], *Gq[QE_MAX_SLOTS], *GqT[QE_MAX_SLOTS];
  // tensor maps: A-role boxes are 128 rows, B-role boxes 256 rows
  CUtensorMap tmXq_A[QE_MAX_SLOTS], tmGq_A[QE_MAX_SLOTS], tmGqT_A[QE_MAX_SLOTS], tmXqT_B[QE_MAX_SLOTS];
  CUtensorMap tmWq_B, tmWqT_B, tmWq_B_mn;
  ActionGraph gF[QE_MAX_SLOTS], gDI[QE_MAX_SLOTS], gDW[QE_MAX_SLOTS], gDWs[QE_MAX_SLOTS], gRefresh, gCommit;
  // QE_CTX_OVERLAP_DW: per slot, "dI of the tape in this slot has been enqueued" / "the dW that released it has"
  cudaEvent_t ev_di[QE_MAX_SLOTS] = {}, ev_dw[QE_MAX_SLOTS] = {};
  bool dw_pending[QE_MAX_SLOTS] = {};
};

namespace {

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

int32_t run_action(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream = nullptr) {
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

}  // namespace
static void destroy_graph(ActionGraph* g) {
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  g->exec = nullptr;
  g->graph = nullptr;
  g->built = false;
}
namespace {

struct Carve {
  uint64_t hist, Wq, WqT, slot0, per_slot, xq, xqT, gq, gqT, total, stage_tk = 0, stage_tn = 0;
};
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
                             float* sinv_dst, int fmt, uint32_t commit_mask = 0) {
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
                        float* sinv_dst, int fmt, uint32_t commit_mask = 0) {
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
void add_forward(qe_layer* L, uint32_t p, const void* x, void* y, std::vector<qe::Launch>& ls, qe_layer* next = nullptr,
                 uint32_t pn = 0, qe::GemmParams* gemm_out = nullptr, qe::QuantParams* cast_out = nullptr) {
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
void add_dI(qe_layer* L, uint32_t p, const void* dy, void* dx, std::vector<qe::Launch>& ls, qe_layer* prev = nullptr,
            uint32_t pp = 0, qe::GemmParams* gemm_out = nullptr, qe::QuantParams* cast_out = nullptr) {
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

// Weight-gradient GEMMs of different layers that follow one another share one launch where the kernel allows it
// (all on the paired variant): the persistent CTAs pack their tiles into common waves and the launch is paid once.
// The layers' gradient slices are disjoint (destination registry), so the GEMMs are independent.
struct DWBatch {
  qe::GemmParams gp[4];
  qe_layer* layer[4];
  uint32_t n = 0;
  bool has(const qe_layer* L) const {
    for (uint32_t i = 0; i < n; ++i)
      if (layer[i] == L) return true;
    return false;
  }
  void flush(qe_ctx* ctx, std::vector<qe::Launch>& ls) {
    qe::GemmParams paired[4];
    uint32_t np = 0;
    for (uint32_t i = 0; i < n; ++i)
      if (qe::gemm_uses_pair(gp[i].M)) paired[np++] = gp[i];
    qe::Launch l;
    const bool grouped = np >= 2 && qe::make_gemm_group(paired, np, ctx->dev->num_sms, &l);
    if (grouped) {
      ls.push_back(l);
      ctx->stats.grouped_dw += np;
    }
    for (uint32_t i = 0; i < n; ++i)
      if (!grouped || !qe::gemm_uses_pair(gp[i].M)) ls.push_back(qe::make_gemm(gp[i], ctx->dev->num_sms));
    n = 0;
  }
  void add(qe_ctx* ctx, qe_layer* L, const qe::GemmParams& g, std::vector<qe::Launch>& ls) {
    if (n == 4 || has(L)) flush(ctx, ls);  // a layer's own GEMMs accumulate into one slice: never in one launch
    gp[n] = g;
    layer[n++] = L;
  }
};

}  // namespace

// ================================================================================================ C ABI
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

// Graph of a launch list identified by a hash (whole steps, multi-layer dW calls); rebuilt when the list's length
// changed under the same key (e.g. no weight refresh this time).
static ActionGraph* keyed_graph(qe_ctx* ctx, uint64_t key, size_t n_launches) {
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

struct Fnv {
  uint64_t key = 1469598103934665603ull;  // FNV-1a
  void mix(const void* ptr, size_t n) {
    const unsigned char* c = (const unsigned char*)ptr;
    for (size_t i = 0; i < n; ++i) key = (key ^ c[i]) * 1099511628211ull;
  }
};

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

static int32_t run_keyed(qe_ctx* ctx, uint64_t key, const std::vector<qe::Launch>& ls) {
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

int32_t qe_run_together(qe_ctx* ctx, qe_action* acts, uint32_t n, float* grad, uint64_t grad_elems, void* caller_stream) {
  TogetherPrep pr;
  int32_t st = together_prepare(ctx, acts, n, grad, grad_elems, &pr);  // check (every action, before anything runs)
  if (st != QE_OK) return st;
  cudaStream_t caller = (cudaStream_t)caller_stream;
  if ((st = handoff_in(ctx, caller)) != QE_OK) return st;
  if (pr.any_dw && ctx->dw_stream) {  // weight gradients issued earlier on the second stream accumulate into the same buffer
    QE_CUDA(cudaEventRecord(ctx->ev_dw_in, ctx->dw_stream));
    QE_CUDA(cudaStreamWaitEvent(ctx->exec_stream, ctx->ev_dw_in, 0));
  }
  std::vector<qe::Launch> ls;
  Fnv h;
  h.mix("together", 9);
  if ((st = together_build(ctx, acts, n, pr, grad, ls, &h)) != QE_OK) return st;
  if ((st = run_keyed(ctx, h.key, ls)) != QE_OK) return st;  // ... run ...
  if (ctx->dw_stream)
    for (uint32_t i = 0; i < n; ++i)
      if (acts[i].kind == QE_ACT_DI) QE_CUDA(cudaEventRecord(acts[i].layer->ev_di[pr.slot[i]], ctx->exec_stream));
  if ((st = handoff_out(ctx, caller)) != QE_OK) return st;
  return together_commit(acts, n, grad, pr);  // ... commit
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
    struct Unit { uint32_t kind, mb, begin, end, done; int prev; };
    std::vector<Unit> units;
    std::vector<uint8_t> taken(n_actions, 0);
    bool ok = true;
    int last_of_kind[3] = {-1, -1, -1};
    for (uint32_t i = 0; i < n_actions && ok; ++i) {
      const qe_step_action& a = actions[i];
      ok = a.kind <= QE_ACT_DW && a.layer < n_layers && a.mb < M;
      if (!ok) break;
      bool fresh = units.empty() || units.back().kind != a.kind || units.back().mb != a.mb;
      for (uint32_t j = fresh ? i : units.back().begin; !fresh && j < i; ++j) fresh = actions[j].layer == a.layer;
      if (fresh) {
        units.push_back(Unit{a.kind, a.mb, i, i, 0, last_of_kind[a.kind]});
        last_of_kind[a.kind] = (int)units.size() - 1;
      }
      units.back().end = i + 1;
    }
    std::vector<uint8_t> issued((size_t)3 * n_layers * M, 0);  // [kind][layer][mb]
    auto was = [&](uint32_t kind, uint32_t layer, uint32_t mb) -> uint8_t& { return issued[((size_t)kind * n_layers + layer) * M + mb]; };
    std::vector<uint32_t> live(n_layers);
    for (uint32_t l = 0; l < n_layers; ++l) live[l] = layers[l]->contract->live_tapes();
    size_t first = 0;
    while (ok && first < units.size()) {
      std::vector<uint32_t> group;
      for (size_t ui = first; ui < units.size() && ui < first + ctx->step_window && group.size() < QE_MAX_TOGETHER; ++ui) {
        const Unit& u = units[ui];
        for (uint32_t i = u.begin; i < u.end && group.size() < QE_MAX_TOGETHER; ++i) {
          if (taken[i]) continue;
          const qe_step_action& a = actions[i];
          bool ready = true;
          for (uint32_t gi : group)  // one action of a kind per layer, never two of one (layer, microbatch)
            ready = ready && !((actions[gi].kind == a.kind && actions[gi].layer == a.layer) || (actions[gi].layer == a.layer && actions[gi].mb == a.mb));
          if (u.prev >= 0) {  // each layer sees the units of a kind in list order
            const Unit& p = units[u.prev];
            for (uint32_t j = p.begin; j < p.end; ++j)
              if (actions[j].layer == a.layer) ready = ready && taken[j] == 2;
          }
          if (a.kind == QE_ACT_F) ready = ready && live[a.layer] < layers[a.layer]->cfg.slots;
          if (a.kind == QE_ACT_DI) ready = ready && was(QE_ACT_F, a.layer, a.mb) == 2;
          if (a.kind == QE_ACT_DW) ready = ready && was(QE_ACT_DI, a.layer, a.mb) == 2;
          if (ready) {
            group.push_back(i);
            taken[i] = 1;
          }
          if (a.kind != QE_ACT_DW) break;  // F and dI: only the unit's next layer can be ready
        }
      }
      if (group.empty()) {
        ok = false;
        break;
      }
      for (uint32_t gi : group) {  // visible to later rounds only
        const qe_step_action& a = actions[gi];
        taken[gi] = 2;
        was(a.kind, a.layer, a.mb) = 2;
        if (a.kind == QE_ACT_F) live[a.layer] += 1;
        if (a.kind == QE_ACT_DW) live[a.layer] -= 1;
      }
      // F and dI actions must be taken in the unit's order: mark "next" by skipping taken ones above; advance `first`
      rounds.push_back(group);
      while (first < units.size()) {
        bool all = true;
        for (uint32_t i = units[first].begin; i < units[first].end; ++i) all = all && taken[i] == 2;
        if (!all) break;
        ++first;
      }
    }
    if (!ok) rounds.clear();
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

// ------------------------------------------------------------------------------------------------ standalone kernels
static int32_t current_device_info(DeviceInfo** d) {
  int dev = 0;
  QE_CUDA(cudaGetDevice(&dev));
  return device_info(dev, d);
}

static int32_t launch_on(const qe::Launch& l, cudaStream_t s) {
  QE_CUDA(launch_pdl(l, s));
  return QE_OK;
}

int32_t qe_quantize(const void* x, uint32_t rows, uint32_t cols, const float* scale_dev, uint32_t fmt, void* q,
                    void* qT, float* amax_dev, void* stream) {
  if (!x || !scale_dev || !q) return fail(QE_ERR_BAD_ARG, "null argument");
  if (fmt > QE_E5M2) return fail(QE_ERR_BAD_ARG, "fp8_format %u", fmt);
  if (rows == 0 || cols == 0 || rows % 64 || cols % 64) return fail(QE_ERR_SHAPE, "rows %u cols %u must be multiples of 64", rows, cols);
  if (((uintptr_t)x & 15u) || ((uintptr_t)q & 7u) || ((uintptr_t)qT & 7u)) return fail(QE_ERR_BAD_ARG, "misaligned pointer");
  qe::QuantParams qp{};
  qp.x = (const uint16_t*)x;
  qp.q = (uint8_t*)q;
  qp.qT = (uint8_t*)qT;
  qp.rows = rows;
  qp.cols = cols;
  qp.scale = scale_dev;
  qp.amax_bits = (uint32_t*)amax_dev;
  qp.fmt = (int32_t)fmt;
  return launch_on(qe::make_quantize(qp), (cudaStream_t)stream);
}

uint32_t qe_amax_partials(void) { return qe::kAmaxPartials; }

int32_t qe_amax(const void* x, uint64_t n, float* partials, float* amax_dev, void* stream) {
  if (!x || !partials || !amax_dev) return fail(QE_ERR_BAD_ARG, "null argument");
  if (n % 8 || ((uintptr_t)x & 15u)) return fail(QE_ERR_SHAPE, "n must be a multiple of 8 and x 16-byte aligned");
  qe::AmaxParams ap{};
  ap.x = (const uint4*)x;
  ap.nvec = n / 8;
  ap.partials = partials;
  ap.out = amax_dev;
  const uint64_t blocks = (ap.nvec + 1023) / 1024;  // 4 vectors per thread per trip
  ap.nparts = (uint32_t)(blocks < 1 ? 1 : blocks > qe::kAmaxPartials ? qe::kAmaxPartials : blocks);
  int32_t st = launch_on(qe::make_amax_pass1(ap), (cudaStream_t)stream);
  if (st != QE_OK) return st;
  return launch_on(qe::make_amax_pass2(ap), (cudaStream_t)stream);
}

int32_t qe_accumulate(float* dst, const float* src, uint64_t n, int32_t accumulate, void* stream) {
  if (!dst || !src) return fail(QE_ERR_BAD_ARG, "null argument");
  if (n % 4 || (((uintptr_t)dst | (uintptr_t)src) & 15u)) return fail(QE_ERR_SHAPE, "n must be a multiple of 4, pointers 16-byte aligned");
  qe::AccumParams ap{};
  ap.dst = (float4*)dst;
  ap.src = (const float4*)src;
  ap.nvec = n / 4;
  ap.accumulate = accumulate;
  return launch_on(qe::make_accumulate(ap), (cudaStream_t)stream);
}

int32_t qe_arena_reduce(const void* views, uint64_t view_elems, uint32_t M, float* dst, void* stream) {
  if (!views || !dst) return fail(QE_ERR_BAD_ARG, "null argument");
  if (M < 1 || M > QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "M %u", M);
  if (view_elems == 0 || view_elems % 8 || (((uintptr_t)views | (uintptr_t)dst) & 15u)) return fail(QE_ERR_BAD_ARG, "views of a multiple of 8 elements, 16-byte aligned");
  qe::ArenaReduceParams ap{};
  ap.views = (const uint4*)views;
  ap.dst = (float4*)dst;
  ap.view_vec = view_elems / 8;
  ap.M = M;
  return launch_on(qe::make_arena_reduce(ap), (cudaStream_t)stream);
}

// Validates one standalone GEMM and fills its parameter block.
static int32_t standalone_gemm(DeviceInfo* dev, const void* a, uint32_t a_fmt, uint32_t a_mn, const void* b, uint32_t b_fmt,
                               uint32_t b_mn, uint32_t M, uint32_t Nn, uint32_t Kc, const float* alpha_a, const float* alpha_b,
                               void* d, uint32_t out_kind, float* amax_dev, uint32_t* status_dev, qe::GemmParams* out) {
  if (!a || !b || !alpha_a || !alpha_b || !d || !status_dev) return fail(QE_ERR_BAD_ARG, "null argument");
  if (a_fmt > QE_E5M2 || b_fmt > QE_E5M2 || out_kind > 2 || a_mn > 1 || b_mn > 1) return fail(QE_ERR_BAD_ARG, "bad enum");
  if (!shape_ok(M) && M != 128) return fail(QE_ERR_SHAPE, "M=%u", M);
  if (!shape_ok(Nn) || (!shape_ok(Kc) && Kc != 128)) return fail(QE_ERR_SHAPE, "N=%u Kc=%u", Nn, Kc);
  if ((a_mn || b_mn) && !qe::gemm_uses_pair(M))
    return fail(QE_ERR_UNSUPPORTED, "MN-major operands need M to be a multiple of 256 (paired-CTA variant), M=%u", M);
  if ((((uintptr_t)a | (uintptr_t)b | (uintptr_t)d) & 15u)) return fail(QE_ERR_BAD_ARG, "misaligned pointer");
  int32_t st;
  qe::GemmParams gp{};
  // contraction-major operand: [rows, Kc]; MN-major operand: [Kc, rows] with a 128 x 128 box
  st = a_mn ? make_map(dev, &gp.tmA, a, Kc, M, 128) : make_map(dev, &gp.tmA, a, M, Kc, 128);
  if (st != QE_OK) return st;
  st = b_mn ? make_map(dev, &gp.tmB, b, Kc, Nn, 128) : make_map(dev, &gp.tmB, b, Nn, Kc, qe::gemm_b_box_rows(M));
  if (st != QE_OK) return st;
  gp.M = M;
  gp.N = Nn;
  gp.Kc = Kc;
  gp.idesc = qe::gemm_idesc((int)a_fmt, (int)b_fmt, M, a_mn != 0, b_mn != 0);
  gp.a_mn = a_mn;
  gp.b_mn = b_mn;
  gp.alpha_a = alpha_a;
  gp.alpha_b = alpha_b;
  gp.out = d;
  gp.ldo = Nn;
  gp.epi = (int32_t)out_kind;
  if ((st = make_out_map(dev, &gp.tmD, d, M, Nn, Nn, out_kind != 0)) != QE_OK) return st;
  gp.amax_bits = (uint32_t*)amax_dev;
  gp.status = status_dev;
  *out = gp;
  return QE_OK;
}

int32_t qe_gemm_fp8_ex(const void* a, uint32_t a_fmt, uint32_t a_mn, const void* b, uint32_t b_fmt, uint32_t b_mn,
                       uint32_t M, uint32_t Nn, uint32_t Kc, const float* alpha_a, const float* alpha_b, void* d,
                       uint32_t out_kind, float* amax_dev, uint32_t* status_dev, void* stream) {
  DeviceInfo* dev = nullptr;
  int32_t st = current_device_info(&dev);
  if (st != QE_OK) return st;
  qe::GemmParams gp;
  if ((st = standalone_gemm(dev, a, a_fmt, a_mn, b, b_fmt, b_mn, M, Nn, Kc, alpha_a, alpha_b, d, out_kind, amax_dev, status_dev, &gp)) != QE_OK) return st;
  return launch_on(qe::make_gemm(gp, dev->num_sms), (cudaStream_t)stream);
}

int32_t qe_gemm_fp8_group(const qe_gemm_desc* descs, uint32_t n, uint32_t* status_dev, void* stream) {
  if (!descs || !status_dev) return fail(QE_ERR_BAD_ARG, "null argument");
  if (n < 2 || n > 8) return fail(QE_ERR_BAD_ARG, "a group holds 2 to 8 problems, got %u", n);
  DeviceInfo* dev = nullptr;
  int32_t st = current_device_info(&dev);
  if (st != QE_OK) return st;
  qe::GemmParams gp[8];
  for (uint32_t i = 0; i < n; ++i) {
    const qe_gemm_desc& q = descs[i];
    if (!qe::gemm_uses_pair(q.M)) return fail(QE_ERR_UNSUPPORTED, "problem %u: M=%u is not a multiple of 256", i, q.M);
    if ((st = standalone_gemm(dev, q.a_dev, q.a_format, q.a_mn, q.b_dev, q.b_format, q.b_mn, q.M, q.Nn, q.Kc, q.alpha_a_dev,
                              q.alpha_b_dev, q.d_dev, q.out_kind, q.amax_dev, status_dev, &gp[i])) != QE_OK)
      return st;
  }
  qe::Launch l;
  if (!qe::make_gemm_group(gp, n, dev->num_sms, &l)) return fail(QE_ERR_UNSUPPORTED, "the problems cannot share a launch");
  return launch_on(l, (cudaStream_t)stream);
}

int32_t qe_gemm_fp8(const void* a, uint32_t a_fmt, const void* b, uint32_t b_fmt, uint32_t M, uint32_t Nn, uint32_t Kc,
                    const float* alpha_a, const float* alpha_b, void* d, uint32_t out_kind, float* amax_dev,
                    uint32_t* status_dev, void* stream) {
  return qe_gemm_fp8_ex(a, a_fmt, 0, b, b_fmt, 0, M, Nn, Kc, alpha_a, alpha_b, d, out_kind, amax_dev, status_dev, stream);
}

}  // extern "C"
