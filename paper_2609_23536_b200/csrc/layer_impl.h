// Internals shared by the translation units of the layer API: the context and layer objects, the launch builders of
// the three actions and the execution layer (eager launches or CUDA graphs, bracketed by the two-way stream handshake).
#pragma once
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

namespace qe_impl {


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceInfo {
  bool ready = false;
  int device = -1, num_sms = 0, cc_major = 0;
  EncodeTiledFn encode = nullptr;
};

int32_t device_info(int device, DeviceInfo** out);
int32_t current_device_info(DeviceInfo** d);
int32_t make_map(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t inner, uint32_t box_rows);
int32_t make_out_map(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t M, uint64_t N, uint64_t ldo, bool fp32);
int32_t make_out_map_u8(const DeviceInfo* d, CUtensorMap* map, const void* ptr, uint64_t M, uint64_t N, uint64_t ld);
inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }
inline bool shape_ok(uint32_t v) { return v >= 256 && v % 128 == 0 && v <= (1u << 20); }

}  // namespace qe_impl
using qe_impl::DeviceInfo;

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

namespace qe_impl {

void destroy_graph(ActionGraph* g);
void ctx_release(qe_ctx* c);

// ---- execution layer
cudaError_t launch_pdl(const qe::Launch& l, cudaStream_t stream);
int32_t launch_on(const qe::Launch& l, cudaStream_t s);
int32_t launch_eager(qe_ctx* ctx, const qe::Launch& l, cudaStream_t stream);
int32_t build_graph(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream);
int32_t replay_graph(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream);
int32_t handoff_in(qe_ctx* ctx, cudaStream_t caller);
int32_t handoff_out(qe_ctx* ctx, cudaStream_t caller);
int32_t host_upload(qe_ctx* ctx, void* dst, const void* src_host, size_t bytes, cudaStream_t caller);
int32_t host_download(qe_ctx* ctx, void* dst_host, const void* src, size_t bytes);
int32_t run_action(qe_ctx* ctx, ActionGraph* g, const std::vector<qe::Launch>& ls, cudaStream_t stream = nullptr);
ActionGraph* keyed_graph(qe_ctx* ctx, uint64_t key, size_t n_launches);
int32_t run_keyed(qe_ctx* ctx, uint64_t key, const std::vector<qe::Launch>& ls);

// ---- workspace and launch builders
struct Carve {
  uint64_t hist, Wq, WqT, slot0, per_slot, xq, xqT, gq, gqT, total, stage_tk = 0, stage_tn = 0;
};
Carve carve(const qe_layer_config& c);
int32_t check_config(const qe_layer_config* c);
qe::CommitParams commit_params(qe_layer* L, uint32_t mask, uint32_t bump, const float* override_amax);
qe::QuantParams quant_params(qe_layer* L, const void* x, uint8_t* q, uint8_t* qT, uint32_t rows, uint32_t cols, int cls,
                             float* sinv_dst, int fmt, uint32_t commit_mask = 0);
qe::Launch quant_launch(qe_layer* L, const void* x, uint8_t* q, uint8_t* qT, uint32_t rows, uint32_t cols, int cls,
                        float* sinv_dst, int fmt, uint32_t commit_mask = 0);
void add_refresh(qe_layer* L, std::vector<qe::Launch>& ls);
void add_forward(qe_layer* L, uint32_t p, const void* x, void* y, std::vector<qe::Launch>& ls, qe_layer* next = nullptr,
                 uint32_t pn = 0, qe::GemmParams* gemm_out = nullptr, qe::QuantParams* cast_out = nullptr);
void add_dI(qe_layer* L, uint32_t p, const void* dy, void* dx, std::vector<qe::Launch>& ls, qe_layer* prev = nullptr,
            uint32_t pp = 0, qe::GemmParams* gemm_out = nullptr, qe::QuantParams* cast_out = nullptr);
qe::GemmParams dW_gemm(qe_layer* L, uint32_t p, float* dst, int32_t accumulate, float* temp);
qe::GemmParams dW_gemm_view(qe_layer* L, uint32_t p, void* view);
void add_dW(qe_layer* L, uint32_t p, float* dst, int32_t accumulate, float* temp, std::vector<qe::Launch>& ls);

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

struct Fnv {
  uint64_t key = 1469598103934665603ull;  // FNV-1a
  void mix(const void* ptr, size_t n) {
    const unsigned char* c = (const unsigned char*)ptr;
    for (size_t i = 0; i < n; ++i) key = (key ^ c[i]) * 1099511628211ull;
  }
};


}  // namespace qe_impl
