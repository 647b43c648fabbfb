/*
 * qe.h -- C ABI of libqe: an FP8 delayed-scaling linear layer run as three checked actions
 * (forward F, input-gradient dI, deferred weight-gradient dW) on one NVIDIA B200 (sm_100a).
 *
 * The operations and their rules follow the QEffect contract:
 *   Eqs. 1-2      TapeKey(e,s,m,u,i) / TapeRef(p,g_p): retained work is named by a logical key and by a slot
 *                 plus its generation; a consumer presents both.
 *   Eqs. 3-5      (Y,S1,T)=F(X,W,S0); (dX,S2,Q)=dI(dY,T,S1); dW=dW(Q).  F and dI advance the effect token and
 *                 the scaling state once each; dW never touches scaling state.
 *   Sec. 3.3      weight version e_W and cache version e_C; the first forward after an optimizer step refreshes
 *                 the quantised-weight cache.
 *   Sec. 3.4      direct gradient placement: dW accumulates in place into a caller-owned flat FP32 buffer.
 *   Algorithm 1   every action is check -> run -> commit; a failed check changes nothing.
 *   Sec. 4.4      capture/replay with a caller->graph wait and a graph->caller completion event on every call.
 *   Invariants 1-4.
 *
 * Conventions
 *   - Every function returns a qe_status (0 = QE_OK, negative = error).  Nothing throws, aborts or exits.
 *     qe_last_error() returns a thread-local, human-readable message for the last failure on this thread.
 *   - "dev" pointers are CUDA device pointers on the context's device; "host" pointers are ordinary host
 *     memory.  The library never frees caller memory.  All device memory a layer uses lives in the workspace
 *     the caller passes to qe_layer_create (size from qe_layer_workspace_bytes); the library itself allocates
 *     no device memory.
 *   - Tensors are dense row-major.  bf16 = IEEE bfloat16 bit patterns (2 bytes).  Tokens T, in-features K,
 *     out-features N:  X[T,K], W[N,K], Y[T,N], dY[T,N], dX[T,K]; a gradient slice is [N,K] FP32 at
 *     grad_buf + offset (offset in ELEMENTS).  T, K, N must be multiples of 128 in [256, 2^20].
 *   - Streams are cudaStream_t passed as void* (NULL = the legacy default stream).  Work is issued on the
 *     context's own execution stream; each action first makes that stream wait on the caller's stream and
 *     finally makes the caller's stream wait on the action's tail, so the caller may use its outputs on
 *     `caller_stream` without further synchronisation (bidirectional completion).
 *   - Device-side waits are bounded; if one expires the kernel sets a status word and returns.  The host reads
 *     that word at qe_optimizer_boundary / qe_get_state and reports QE_ERR_TIMEOUT.
 */
#ifndef QE_H_
#define QE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum qe_status {
  QE_OK = 0,
  QE_ERR_BAD_ARG = -1,      /* null pointer, index out of range, unknown enum value                           */
  QE_ERR_SHAPE = -2,        /* T, K or N not a multiple of 128 or outside [256, 2^20]                         */
  QE_ERR_KEY_LIVE = -3,     /* forward: the same TapeKey already has a live tape (mapping must stay injective)*/
  QE_ERR_POOL_FULL = -4,    /* forward: no free slot; an occupied slot is never pre-empted                    */
  QE_ERR_STALE_CACHE = -5,  /* forward: e_C != e_W on a non-first forward ("cache refresh required")          */
  QE_ERR_ABORTED = -6,      /* the step was aborted; the arena is unusable until qe_arena_rebuild             */
  QE_ERR_STALE_REF = -7,    /* the reference's generation does not name the slot's live tape                  */
  QE_ERR_KEY_MISMATCH = -8, /* the slot is live with that generation but under a different key               */
  QE_ERR_EPOCH = -9,        /* caller's weight version, or the tape's epoch, differs from e_W                 */
  QE_ERR_DUP_CONSUME = -10, /* dI (or dW) already consumed this tape                                          */
  QE_ERR_ORDER = -11,       /* dW before dI; or first gradient write of an epoch is not microbatch 0          */
  QE_ERR_DEST = -12,        /* destination null/misaligned/too small/not the bound one/aliasing another layer */
  QE_ERR_DUP_WRITE = -13,   /* this microbatch already wrote its gradient in this epoch                       */
  QE_ERR_PENDING = -14,     /* live tape at a quiescent point (optimizer boundary, checkpoint, rebuild)       */
  QE_ERR_INCOMPLETE = -15,  /* optimizer boundary: some configured microbatch has not written its gradient    */
  QE_ERR_CUDA = -16,        /* a CUDA runtime/driver call failed (message has the CUDA error string)          */
  QE_ERR_TIMEOUT = -17,     /* a bounded device-side wait expired (device status word non-zero)               */
  QE_ERR_WORKSPACE = -18,   /* workspace null, misaligned (256 B) or smaller than qe_layer_workspace_bytes    */
  QE_ERR_UNSUPPORTED = -19  /* no sm_100 device, or a size beyond a stated maximum                            */
} qe_status;

typedef enum qe_exec_mode { QE_EXEC_EAGER = 0, QE_EXEC_GRAPH = 1 } qe_exec_mode;
typedef enum qe_tensor_class { QE_CLASS_X = 0, QE_CLASS_W = 1, QE_CLASS_G = 2, QE_CLASS_Y = 3 } qe_tensor_class;
typedef enum qe_fp8_format { QE_E4M3 = 0, QE_E5M2 = 1 } qe_fp8_format;

#define QE_MAX_SLOTS 64u
#define QE_MAX_MICROBATCHES 64u
#define QE_MAX_HISTORY 4096u
#define QE_INVALID_EPOCH UINT64_MAX

/* ---- Eq. 1 / Eq. 2 ------------------------------------------------------------------------------------------- */
typedef struct qe_tape_key { uint32_t epoch, stage, mb, unit, inv; } qe_tape_key; /* (e, s, m, u, i)              */
typedef struct qe_tape_ref { uint32_t slot; uint32_t reserved; uint64_t gen; } qe_tape_ref; /* (p, g_p)          */
/* The (K, R) pair carried on the saved-value edge (Sec. 4.2).  Returned by value, owned by the caller, meaningless
 * after the slot is released: a later use fails with QE_ERR_STALE_REF and never touches the slot's new occupant. */
typedef struct qe_tape { qe_tape_key key; uint32_t reserved; qe_tape_ref ref; } qe_tape;

/* ================================================================================================================
 * Contract core (host only; creates no CUDA context).  The layer calls use it internally with exactly these
 * check/commit pairs; it is exported so that the contract can be exercised without a GPU (Table 3: the fault
 * injections run in a process that initialises no CUDA context).
 * ============================================================================================================== */
typedef struct qe_contract qe_contract;
typedef struct qe_registry qe_registry; /* gradient destinations bound this epoch by a group of layers (alias check) */

int32_t qe_registry_create(qe_registry** out);
/* Contracts created with a registry share ownership of it; the handle may be destroyed before or after them. */
int32_t qe_registry_destroy(qe_registry*);

/* slots in [1, QE_MAX_SLOTS]; registry may be NULL (then only this layer's own rules are checked). */
int32_t qe_contract_create(uint32_t slots, uint32_t stage, uint32_t unit, uint32_t inv, qe_registry* registry,
                           qe_contract** out);
int32_t qe_contract_destroy(qe_contract*);

/* Forward (Algorithm 1, forward branch).  check: aborted? mb < 64? gen == e_W? cache fresh (or first forward of the
 * epoch -> *refresh_out = 1)? key not live? free slot (lowest index -> *slot_out)?  commit: occupy the slot,
 * g_p += 1, e_C <- e_W on refresh, token += 1; writes the tape. */
int32_t qe_contract_forward_check(const qe_contract*, uint32_t mb, uint64_t gen, int32_t* refresh_out,
                                  uint32_t* slot_out);
int32_t qe_contract_forward_commit(qe_contract*, uint32_t mb, qe_tape* tape_out);
/* Input gradient (Algorithm 1, input-grad branch).  check: generation, key, epoch, dI bit clear.  commit: set dI bit, token += 1. */
int32_t qe_contract_dI_check(const qe_contract*, const qe_tape*);
int32_t qe_contract_dI_commit(qe_contract*, const qe_tape*);
/* Weight gradient (Algorithm 1, weight-grad branch).  dest_addr = address of element 0 of the flat buffer, as an integer.  check:
 * resolve; dW bit clear; dI bit set; destination valid (non-null, dest_addr + 4*offset 16-byte aligned,
 * offset + slice_elems <= dest_elems, equal to the destination bound this epoch, no overlap with another
 * layer's bound slice); this microbatch has not written; the first write of the epoch is microbatch 0.
 * *accumulate_out = 0 for the first write of the epoch (overwrite), 1 afterwards.  commit: bind destination, set
 * mask bit and dW bit, release the slot (generation kept). */
int32_t qe_contract_dW_check(const qe_contract*, const qe_tape*, uint64_t dest_addr, uint64_t dest_elems,
                             uint64_t offset, uint64_t slice_elems, int32_t* accumulate_out);
int32_t qe_contract_dW_commit(qe_contract*, const qe_tape*, uint64_t dest_addr, uint64_t offset,
                              uint64_t slice_elems);
/* Optimizer commit (Algorithm 1, after the loop): no live tape (else PENDING), every microbatch in [0, expected) wrote exactly
 * once (else INCOMPLETE); then e_W += 1, mask cleared, next forward refreshes the cache. */
int32_t qe_contract_boundary(qe_contract*, uint32_t microbatches_expected);
/* The checks of qe_contract_boundary alone (nothing changes): lets a caller that commits several layers together
 * make every layer's check before the first commit. */
int32_t qe_contract_boundary_check(const qe_contract*, uint32_t microbatches_expected);
/* Failure boundary (Sec. 4.5): purge this epoch's tapes (generations kept), mark the arena unusable. */
int32_t qe_contract_abort(qe_contract*);
/* Make the arena usable again after an abort; the epoch restarts with nothing written (PENDING if a tape lives). */
int32_t qe_contract_rebuild(qe_contract*);
/* Mark the quantised-weight cache stale (e_C <- invalid). */
int32_t qe_contract_invalidate_cache(qe_contract*);
/* Invariant 4: QE_OK only when no tape is live ("checkpoint withheld" otherwise -> PENDING). */
int32_t qe_contract_checkpoint_check(const qe_contract*);
/* Restart rule (Algorithm 1, last line; Sec. 3.5): adopt the saved weight version, invalidate the cache so the first
 * forward refreshes it, clear the write mask and the aborted flag.  Process-local identities (slot generations, the
 * effect token) are NOT restored: they keep counting from wherever this process is.  PENDING if a tape is live. */
int32_t qe_contract_restore(qe_contract*, uint64_t e_W);

typedef struct qe_slot_view { uint64_t gen; uint32_t live; uint32_t bits; qe_tape_key key; uint32_t reserved; } qe_slot_view;
typedef struct qe_contract_view {
  uint64_t e_W, e_C, token, write_mask;
  uint32_t fwd_in_epoch, aborted, slots, live_tapes;
  qe_slot_view slot[QE_MAX_SLOTS];
} qe_contract_view;
int32_t qe_contract_get(const qe_contract*, qe_contract_view* out);

/* ================================================================================================================
 * Layer API (CUDA, sm_100a)
 * ============================================================================================================== */
typedef struct qe_ctx qe_ctx;
typedef struct qe_layer qe_layer;

typedef struct qe_ctx_config {
  uint32_t exec_mode; /* qe_exec_mode: launch kernels one by one, or replay one prebuilt CUDA graph per (action, slot) */
  int32_t device;     /* CUDA device ordinal                                                                           */
  void* exec_stream;  /* NULL: the context creates and owns its execution stream (actions then hand off to and from
                         the caller's stream with events).  Non-NULL: a caller-owned cudaStream_t the context executes
                         on; an action called with that same stream as caller_stream needs no event handoff, stream
                         order gives both directions of the completion guarantee.                                     */
  uint32_t flags;     /* QE_CTX_* bits                                                                                 */
  uint32_t step_window; /* qe_step_run: how many units of the list it looks ahead when it cuts the list into rounds of
                         independent actions (0: default 4; 1: action by action, only consecutive dW grouped)         */
  uint32_t reserved[2];
} qe_ctx_config;
/* Run the deferred weight-gradient actions on a second, lower-priority stream of the context so that their
 * thread blocks fill SMs the forward / input-gradient kernels leave idle (dW never touches scaling state, which is
 * what makes it deferrable: Eq. 5, Invariant 1).  Ordering kept by events: dW(m) after dI(m); a slot's next forward
 * after the dW that released it; all dW of a layer in issue order on the one stream (so the accumulation order, and
 * with it every bit of the gradient buffer, is the same as without the flag).  With this flag qe_backward_dW does
 * NOT make the caller's stream wait for the dW: the gradient buffer is complete after qe_optimizer_boundary (which
 * waits for both streams), matching the rule that the optimizer commit requires all arena writes resolved. */
#define QE_CTX_OVERLAP_DW 1u
/* DIAGNOSTIC ONLY -- reproduces the defective one-way handoff of Sec. 2.3 so that it can be measured against the
 * two-way protocol: the execution stream still waits for the caller, but the caller's stream is NOT made to wait for
 * the action's tail.  A consumer on the caller's stream then reads outputs and state before the action has finished
 * (stale data; no fault).  Never set this outside that experiment.  Ignored when the context executes on the
 * caller's own stream. */
#define QE_CTX_UNSAFE_ONE_WAY_HANDOFF 2u

typedef struct qe_layer_config {
  uint32_t T, K, N;       /* tokens, in-features, out-features: multiples of 128 in [256, 2^20]          */
  uint32_t history_len;   /* H in [1, QE_MAX_HISTORY]                                                        */
  int32_t margin;         /* scale = fp8_max / max(history) / 2^margin; margin in [-32, 32]                  */
  uint32_t slots;         /* tape slots P in [1, QE_MAX_SLOTS]                                               */
  uint32_t stage, unit, inv; /* s, u, i of Eq. 1                                                             */
  uint32_t host_io;       /* 1: reserve staging buffers in the workspace for qe_forward_host / qe_backward_dI_host    */
  const void* weight_dev; /* bf16 W[N,K]; caller-owned; read on the first forward of every epoch             */
  uint64_t reserved1[4];
} qe_layer_config;

int32_t qe_ctx_create(const qe_ctx_config*, qe_ctx** out);
/* A context stays alive until it has been destroyed AND its last layer has been destroyed (either order). */
int32_t qe_ctx_destroy(qe_ctx*);
int32_t qe_layer_workspace_bytes(const qe_layer_config*, uint64_t* bytes_out);
/* workspace_dev: 256-byte aligned device memory of at least qe_layer_workspace_bytes; owned by the caller, must
 * outlive the layer.  The call zero-initialises the state in it (histories 0, scales 1) on the execution stream, so
 * the memory must have no work pending on any other stream when the call is made (memory fresh from a stream-ordered
 * allocator may still be written by kernels that used it before it was freed: synchronise that stream first). */
int32_t qe_layer_create(qe_ctx*, const qe_layer_config*, void* workspace_dev, uint64_t workspace_bytes,
                        qe_layer** out);
int32_t qe_layer_destroy(qe_layer*);

/* F (Eq. 3).  x_dev bf16 [T,K] in, y_dev bf16 [T,N] out.  `gen` is the caller's view of the weight version and must
 * equal e_W.  On the first forward of an epoch the weight is re-quantised (E4M3; plus its transpose where dI needs one) and its amax
 * committed.  Then: X quantised to E4M3 with the current scale (amax taken in the same pass; the inverse scale is
 * snapshotted into the tape slot), Y = bf16((Xq Wq^T) * sinv_X * sinv_W) on the tensor cores with max|Y| reduced in
 * the epilogue, and the X and Y histories/scales updated.  *tape_out names the retained work. */
int32_t qe_forward(qe_layer*, uint32_t mb, uint64_t gen, const void* x_dev, void* y_dev, void* caller_stream,
                   qe_tape* tape_out);
/* dI (Eq. 4).  dy_dev bf16 [T,N] in, dx_dev bf16 [T,K] out.  Quantises dY to E5M2 (and, where dW needs it, its transpose, retained for
 * dW), dX = bf16((Gq Wq) * sinv_G * sinv_W), commits the gradient amax/scale once. */
int32_t qe_backward_dI(qe_layer*, const qe_tape*, const void* dy_dev, void* dx_dev, void* caller_stream);
/* F and dI with HOST buffers (layer created with host_io = 1).  The input is copied host-to-device into the layer's
 * fixed staging buffer after the caller->execution edge (the dynamic-input copy of Sec. 4.4), the action runs on
 * the staging buffers -- in graph mode the graph's addresses therefore never change -- and the output is copied
 * device-to-host before the execution->caller edge, so it is complete for work the caller queues after the call (or
 * after synchronising caller_stream on the host).  The two copies run on copy streams of the context, ordered with
 * the execution stream by events: the upload of a call overlaps the read-back of the call before it (the host link
 * is full duplex), the kernels wait for both.  Pinned host memory makes the copies asynchronous; y_host / dx_host
 * may be NULL to skip the read-back.  Same checks, state transitions and results as qe_forward / qe_backward_dI. */
int32_t qe_forward_host(qe_layer*, uint32_t mb, uint64_t gen, const void* x_host, void* y_host, void* caller_stream,
                        qe_tape* tape_out);
int32_t qe_backward_dI_host(qe_layer*, const qe_tape*, const void* dy_host, void* dx_host, void* caller_stream);
/* dW (Eq. 5) with direct gradient placement (Sec. 3.4).  D = (Gq^T Xq) * sinv_G * sinv_X using the inverse scales
 * snapshotted in the tape; grad_buf_dev[offset + n*K + k] = D (first write of the epoch) or += D (FP32, in place:
 * one round-to-nearest addition per element and call, performed in L2 by a bulk tensor reduction, subnormal values
 * kept; deterministic, calls ordered by the stream).  No staging copy, no scale-state change. */
int32_t qe_backward_dW(qe_layer*, const qe_tape*, float* grad_buf_dev, uint64_t grad_buf_elems, uint64_t offset,
                       void* caller_stream);
/* The copied-gradient comparison path of Sec. 3.4: same checks and the same final values, but D is first written
 * to temp_dev (FP32 [N,K], caller-owned scratch) and then added into the destination by a second kernel. */
int32_t qe_backward_dW_staged(qe_layer*, const qe_tape*, float* grad_buf_dev, uint64_t grad_buf_elems,
                              uint64_t offset, float* temp_dev, void* caller_stream);
/* F of one layer and dI of another in one call (Sec. 4.2: in the steady state of a split-backward schedule a stage
 * holds a forward unit and an input-gradient unit at once; their chains through the layers are independent).  The
 * same checks, results (bit for bit) and state transitions as qe_forward(layer_f, mb, gen, x_dev, y_dev, stream,
 * tape_out) followed by qe_backward_dI(layer_b, tape_b, dy_dev, dx_dev, stream), with the two GEMMs in one kernel
 * launch where both can run on the paired-CTA variant (T a multiple of 256).  layer_f != layer_b, one context.  Both
 * checks are made before anything runs: on a contract error nothing ran and neither layer's state changed. */
int32_t qe_forward_dI_pair(qe_layer* layer_f, uint32_t mb, uint64_t gen, const void* x_dev, void* y_dev,
                           qe_tape* tape_out, qe_layer* layer_b, const qe_tape* tape_b, const void* dy_dev,
                           void* dx_dev, void* caller_stream);
/* Several independent actions in one call (the general form of qe_forward_dI_pair and qe_backward_dW_multi): in
 * the steady state of a split-backward schedule a stage holds a forward unit, an input-gradient unit and a deferred
 * weight-gradient unit at once (Sec. 4.2), none of which depends on another.  The result -- outputs, gradient
 * buffer, scale state, tapes -- is bit for bit that of issuing the actions one after the other in the order given;
 * all GEMMs that can run on the paired-CTA variant share one kernel launch (forward and input-gradient tiles
 * first, weight-gradient tiles after them).  1 <= n <= QE_MAX_TOGETHER; at most one
 * action of a kind per layer; a dW action's tape must already have had its dI (ORDER otherwise, also when that dI
 * is part of the same call).  Every check is made before anything runs, against the state before the call: on a
 * contract error nothing ran and no state changed; in particular a forward cannot take the slot that a dW of the same
 * call is about to release (POOL_FULL if no other slot is free), and the slot a tape lands in may differ from the
 * one-by-one order.  Everything runs on the execution stream (weight gradients issued earlier on the context's second
 * stream are waited for). */
#define QE_MAX_TOGETHER 8
typedef struct qe_action {
  uint32_t kind;          /* QE_ACT_F, QE_ACT_DI or QE_ACT_DW                                                */
  uint32_t mb;            /* F: microbatch                                                                   */
  uint64_t gen;           /* F: the caller's view of the weight version                                      */
  qe_layer* layer;
  const void* in_dev;     /* F: x bf16 [T,K]; dI: dy bf16 [T,N]; dW: unused                                  */
  void* out_dev;          /* F: y bf16 [T,N]; dI: dx bf16 [T,K]; dW: unused                                  */
  qe_tape* tape;          /* F: receives the tape; dI, dW: the tape to consume                               */
  uint64_t grad_offset;   /* dW: element offset of the layer's slice in grad_buf_dev                         */
} qe_action;
int32_t qe_run_together(qe_ctx*, qe_action* actions, uint32_t n, float* grad_buf_dev, uint64_t grad_buf_elems,
                        void* caller_stream);
/* The same with HOST buffers for the F and dI actions (layers created with host_io = 1): in_dev / out_dev then hold
 * host pointers (out may be NULL to skip the read-back); every input is uploaded into its layer's staging buffer
 * first, the kernels run on the staging buffers, the outputs are read back afterwards -- copies on the context's
 * two copy streams as in qe_forward_host, so the uploads of a call overlap the read-backs of the call before it. */
int32_t qe_run_together_host(qe_ctx*, qe_action* actions, uint32_t n, float* grad_buf_dev, uint64_t grad_buf_elems,
                             void* caller_stream);
/* FP8 hand-off between directly chained linears (layers[i+1] consumes layers[i]'s output: same T,
 * K_{i+1} = N_i; host array of n <= QE_MAX_CHAIN distinct layers of one context).  qe_forward_chain runs F of every
 * layer for microbatch mb: x_dev bf16 [T, K_0] in, y_dev bf16 [T, N_{n-1}] out, tapes_out[n].  The output of
 * layers[i] (i < n-1) is never stored as bf16: its forward GEMM's epilogue rounds it to bf16, takes max|Y| of the
 * rounded values (committed as layers[i]'s Y amax and layers[i+1]'s X amax), multiplies by layers[i+1]'s current X
 * scale in FP32 and converts to E4M3 straight into layers[i+1]'s tape slot, with that layer's inverse-scale
 * snapshot -- exactly the bytes and state that qe_forward(layers[i]) followed by qe_forward(layers[i+1]) on the
 * bf16 tensor would have produced, without the cast kernel and its 3 bytes per element.  qe_backward_dI_chain is
 * the same in the backward direction (tapes[] in layer order): dy_dev bf16 [T, N_{n-1}] in, dx_dev bf16 [T, K_0]
 * out, each input gradient handed to the layer before it as E5M2 with that layer's G scale.  Every layer's contract
 * check is made before anything runs; dW of each layer follows through qe_backward_dW / _multi as usual.
 * UNSUPPORTED when a receiving layer keeps transposed FP8 copies (T and N multiples of 256 are required). */
#define QE_MAX_CHAIN 16
int32_t qe_forward_chain(qe_layer* const* layers, uint32_t n, uint32_t mb, uint64_t gen, const void* x_dev,
                         void* y_dev, void* caller_stream, qe_tape* tapes_out);
int32_t qe_backward_dI_chain(qe_layer* const* layers, const qe_tape* tapes, uint32_t n, const void* dy_dev,
                             void* dx_dev, void* caller_stream);
/* The arena as the paper sizes it (Sec. 3.4; capacity A_r = M * sum of sizeof(W)): one bf16 view per matrix
 * parameter and configured microbatch.  arena_dev: bf16 elements; the layer's region is
 * [layer_offset, layer_offset + microbatches * N*K), microbatch m's view starts at layer_offset + m * N*K.
 * qe_backward_dW_arena: same checks, order rules (microbatch 0 first, each microbatch exactly once, destination =
 * the layer's region, bound for the epoch and alias-checked against other layers) and state transitions as
 * qe_backward_dW, but view[n*K + k] = bf16(D) and nothing is accumulated.  layer_offset a multiple of 8.
 * qe_arena_finalize: before the optimizer boundary, grad_buf_dev[offset + i] = sum over m of view_m[i], added in
 * FP32 in microbatch order (one kernel, (2M + 4) bytes per element); INCOMPLETE unless every microbatch wrote,
 * DEST unless the region is the one bound this epoch; changes no contract state.
 * qe_arena_reduce: that kernel alone (views_dev: M contiguous views of view_elems bf16 each, view_elems a multiple
 * of 8, 16-byte aligned). */
int32_t qe_backward_dW_arena(qe_layer*, const qe_tape*, void* arena_dev, uint64_t arena_elems, uint64_t layer_offset,
                             uint32_t microbatches, void* caller_stream);
int32_t qe_arena_finalize(qe_layer*, const void* arena_dev, uint64_t arena_elems, uint64_t layer_offset,
                          uint32_t microbatches, float* grad_buf_dev, uint64_t grad_buf_elems, uint64_t offset,
                          void* caller_stream);
int32_t qe_arena_reduce(const void* views_dev, uint64_t view_elems, uint32_t M, float* dst_dev, void* stream);
/* The W action of Sec. 4.2 for several layers of the stage at once (typically one microbatch's deferred weight
 * gradients): the same checks, results (bit for bit) and state transitions as qe_backward_dW(layers[i], &tapes[i],
 * grad_buf_dev, grad_buf_elems, offsets[i], stream) for i = 0..n-1, but the GEMMs of up to four layers at a time share one
 * kernel launch where each of them can run on the paired-CTA variant (N_i a multiple of 256); the others are
 * launched one by one inside the same call.  layers[] (host array) distinct and of one context, 1 <= n <=
 * QE_MAX_MULTI_DW; tapes[] and offsets[] host arrays of n entries.  All n checks are made before anything runs: on
 * a contract error nothing ran and no layer's state changed.  A bounded wait that expires inside a shared launch
 * is recorded in the status word of every layer that has a GEMM in that launch. */
#define QE_MAX_MULTI_DW 16
int32_t qe_backward_dW_multi(qe_layer* const* layers, const qe_tape* tapes, uint32_t n, float* grad_buf_dev,
                             uint64_t grad_buf_elems, const uint64_t* offsets, void* caller_stream);
/* Optimizer boundary: waits for the execution stream, reads the device status word, then applies
 * qe_contract_boundary (bumping the weight version so that the next forward refreshes the cache). */
int32_t qe_optimizer_boundary(qe_layer*, uint32_t microbatches_expected);
/* The optimizer boundary of n layers of ONE context in one call (Algorithm 1's commit after the loop, for a whole
 * stage): the context's streams are drained once, one small kernel ORs the layers' device status words together and
 * one 4-byte copy brings the result to the host -- where n separate qe_optimizer_boundary calls pay n drains and n
 * blocking copies.  Then every layer's contract check is made (no live tape, every microbatch wrote exactly once)
 * and, only if all n pass, every layer's weight version is bumped.  On any error (QE_ERR_TIMEOUT from a status word,
 * a contract error of some layer) no layer's state has changed.  layers[]: host array of 1 <= n <= 4096 distinct
 * layers. */
int32_t qe_optimizer_boundary_all(qe_layer* const* layers, uint32_t n, uint32_t microbatches_expected);
/* The scale update as a standalone call: push *amax_dev (one FP32 on the device) into the class's history ring and
 * recompute scale = fp8_max / max(history) / 2^margin and its inverse (unchanged if the maximum is 0 or not
 * finite; +Inf clamps to FLT_MAX).  Same kernel F and dI use.  Does not advance the effect token. */
int32_t qe_scale_commit(qe_layer*, uint32_t tensor_class, const float* amax_dev, void* caller_stream);
int32_t qe_abort_step(qe_layer*);
int32_t qe_arena_rebuild(qe_layer*);
int32_t qe_invalidate_cache(qe_layer*);
/* Slot the next successful qe_forward will occupy (lowest free index), or QE_ERR_POOL_FULL. */
int32_t qe_next_slot(const qe_layer*, uint32_t* slot_out);

/* ---- A whole list of actions in one call (host loop in native code; in graph mode ONE graph for the whole list) ---
 * Equivalent to calling qe_forward / qe_backward_dI / qe_backward_dW (or _staged when temp_dev is non-NULL) for
 * actions[0..n) in order, each with gen = its layer's current weight version; the tapes are kept inside the call.
 * All layers must belong to ctx.  io[layer * microbatches + mb] holds the device pointers of that unit (x, y for F;
 * dy, dx for dI).  Layer l's gradient slice is grad_buf_dev + offsets[l].  Every action is checked and committed on
 * the host exactly like the single calls; the kernels of the whole list are then issued behind ONE caller->execution
 * wait and ONE execution->caller event: in eager mode as plain launches, in graph mode as one captured graph that is
 * cached per (layers, actions) and replayed, with kernel-node parameters patched where pointers or the accumulate flag
 * differ from the previous replay.  dW runs on the execution stream here (QE_CTX_OVERLAP_DW does not apply).
 * Independent actions share launches, with bit-identical results (only the slot a tape lands in may differ from the
 * one-by-one order).  The list is read as units -- runs of actions of one kind and microbatch over distinct layers: a
 * forward, input-gradient or weight-gradient unit of the stage -- and cut into rounds of up to QE_MAX_TOGETHER actions
 * whose predecessors were issued in earlier rounds (the previous layer of the own unit for F and dI, the same layer of
 * the previous unit of the kind, F before dI before dW of a (layer, microbatch), a free tape slot), looking
 * qe_ctx_config.step_window units ahead of the earliest unfinished one; a round is issued as qe_run_together would.
 * With temp_dev, with step_window 1, or when the list admits no such plan, actions go one by one and only
 * consecutive dW actions of different layers share launches (as in qe_backward_dW_multi).
 * (The plan honours dependencies, not positions: an action listed before a predecessor that lies within the look-ahead
 * simply runs after it.)
 * If a check fails at action k (the first action of the failing round), the kernels issued so far still run (device and host state stay in step),
 * then every layer of the list is aborted as at a failure boundary (Sec. 4.5) and the failing check's status is
 * returned; qe_arena_rebuild restarts the epoch. */
typedef struct qe_step_action { uint32_t kind; uint32_t layer; uint32_t mb; uint32_t reserved; } qe_step_action;
enum { QE_ACT_F = 0, QE_ACT_DI = 1, QE_ACT_DW = 2 };
typedef struct qe_step_io { const void* x_dev; void* y_dev; const void* dy_dev; void* dx_dev; } qe_step_io;
int32_t qe_step_run(qe_ctx* ctx, qe_layer* const* layers, uint32_t n_layers, const qe_step_action* actions,
                    uint32_t n_actions, uint32_t microbatches, const qe_step_io* io, float* grad_buf_dev,
                    uint64_t grad_buf_elems, const uint64_t* offsets, float* temp_dev, void* caller_stream);
/* The issue plan qe_step_run makes, as host logic of its own (no device needed): cuts actions[0..n) into rounds as
 * described above.  slots[l]: tape slots of layer l; live_now[l]: tapes of layer l alive before the list (NULL: none);
 * window >= 1 units of look-ahead; max_group actions per round.  round_of_action[i] receives the round of action i
 * (rounds are numbered from 0 in issue order), *n_rounds_out their number.  ORDER if the list admits no plan (an
 * action whose predecessors never become ready, or a pool too small), BAD_ARG for a malformed action. */
int32_t qe_plan_rounds(const qe_step_action* actions, uint32_t n_actions, uint32_t n_layers, uint32_t microbatches,
                       const uint32_t* slots, const uint32_t* live_now, uint32_t window, uint32_t max_group,
                       uint32_t* round_of_action, uint32_t* n_rounds_out);


typedef struct qe_class_state {
  float scale, scale_inv;
  uint32_t count;      /* commits so far */
  uint32_t reserved;
} qe_class_state;
typedef struct qe_state_view {
  qe_class_state cls[4];       /* indexed by qe_tensor_class                                                   */
  float cache_sinv_W;          /* inverse weight scale snapshotted when the cache was last refreshed           */
  uint32_t device_status;      /* 0 = clean                                                                    */
  uint64_t device_token;       /* effect token as counted on the device (F and dI kernels' commits)            */
  qe_contract_view contract;   /* host-side bookkeeping (its token must equal device_token)                    */
} qe_state_view;
/* Synchronises the execution stream and copies the state out.  window_out (host, may be NULL): 4*H floats, class c's
 * history at [c*H, (c+1)*H) as a logical window, newest first.  slot_sinv_out (host, may be NULL): 2*P floats,
 * sinv_X of slot p at [p], sinv_G at [P+p]. */
int32_t qe_get_state(qe_layer*, qe_state_view* out, float* window_out, float* slot_sinv_out);
/* Copies a slot's retained FP8 bytes to host memory (testing aid; synchronises).  which: 0 = Xq [T,K],
 * 1 = Xq^T [K,T], 2 = Gq [T,N], 3 = Gq^T [N,T], 4 = Wq [N,K] (slot ignored), 5 = Wq^T [K,N] (slot ignored).
 * Transposed copies exist only where a GEMM needs them: Wq^T when T is not a multiple of 256, Xq^T and Gq^T when N
 * is not (otherwise the tensor cores read the row-major tensor as an MN-major operand) -- QE_ERR_UNSUPPORTED if absent. */
int32_t qe_read_fp8(qe_layer*, uint32_t which, uint32_t slot, void* host_out, uint64_t bytes);

/* Quiescent checkpoint (Sec. 3.5, Invariant 4).  The payload holds PERSISTENT state only: the static configuration
 * (T, K, N, H, margin), the four amax histories with their commit counts, scales and inverse scales, and the weight
 * version e_W.  Graphs, streams, events, slot generations, the effect token, buffer addresses and the quantised-weight
 * cache contents are process-local and are not saved.  qe_state_save waits for the layer's streams, then fails with
 * QE_ERR_PENDING ("checkpoint withheld") while any tape is live.  qe_state_load (into a layer of the same
 * configuration, no live tape) restores the numerics and e_W and invalidates the weight cache, so the first forward
 * after it re-quantises the weight.  host buffers; bytes must equal qe_state_bytes. */
int32_t qe_state_bytes(const qe_layer*, uint64_t* bytes_out);
int32_t qe_state_save(qe_layer*, void* host_out, uint64_t bytes);
int32_t qe_state_load(qe_layer*, const void* host_in, uint64_t bytes);

typedef struct qe_stats {
  uint64_t graphs_built, graph_replays, eager_launches, handoffs, node_param_updates;
  uint64_t kernels_launched;   /* kernels of this library enqueued (eager launches + kernel nodes replayed)   */
  double capture_host_ms;      /* host time spent building graphs                                             */
  uint64_t workspace_bytes;    /* sum over live layers                                                        */
  uint64_t grouped_dw;         /* weight-gradient GEMMs that shared a launch with other layers' (built launches)  */
  uint64_t paired_f_di;        /* forward / input-gradient GEMM pairs that shared a launch                     */
} qe_stats;
int32_t qe_get_stats(const qe_ctx*, qe_stats* out);

/* ================================================================================================================
 * Standalone kernels of the path (no layer state; everything on `stream`)
 * ============================================================================================================== */
/* Fused cast: q[r,c] = fp8_rne_satfinite(fp32(x[r,c]) * *scale_dev); optional transposed copy qT[c,r]; optional
 * amax: *amax_dev = max(*amax_dev, max|x|) (atomic max on the non-negative FP32 bit pattern -- zero it first for a
 * fresh maximum).  rows and cols multiples of 64.  x bf16; q, qT bytes.  qT_dev and amax_dev may be NULL. */
int32_t qe_quantize(const void* x_dev, uint32_t rows, uint32_t cols, const float* scale_dev, uint32_t fp8_format,
                    void* q_dev, void* qT_dev, float* amax_dev, void* stream);
/* max|x| over n bf16 values, two passes without atomics: per-block partial maxima into partials_dev (FP32, at least
 * qe_amax_partials() entries, scratch owned by the caller), then a final block writes *amax_dev.  n multiple of 8. */
int32_t qe_amax(const void* x_dev, uint64_t n, float* partials_dev, float* amax_dev, void* stream);
uint32_t qe_amax_partials(void);
/* dst[i] (=|+=) src[i] in FP32 (the second half of the copied-gradient path).  n multiple of 4, 16-byte aligned. */
int32_t qe_accumulate(float* dst_dev, const float* src_dev, uint64_t n, int32_t accumulate, void* stream);
/* One FP8 GEMM on the tensor cores: D[m,n] = (sum_k A[m,k] B[n,k]) * *alpha_a_dev * *alpha_b_dev with A [M,Kc] and
 * B [Nn,Kc] both contraction-major bytes.  out_kind 0: bf16 D (amax_dev optional, as in qe_quantize); 1: FP32
 * D overwrite; 2: FP32 D accumulate.  M, Kc multiples of 128 (>= 128), Nn a multiple of 128 (>= 256).  A 256-row paired-CTA variant runs when
 * M is a multiple of 256, a single-CTA 128-row variant otherwise.  status_dev: one uint32 the kernel ORs error
 * bits into (caller zeroes it). */
int32_t qe_gemm_fp8(const void* a_dev, uint32_t a_format, const void* b_dev, uint32_t b_format, uint32_t M,
                    uint32_t Nn, uint32_t Kc, const float* alpha_a_dev, const float* alpha_b_dev, void* d_dev,
                    uint32_t out_kind, float* amax_dev, uint32_t* status_dev, void* stream);

/* As qe_gemm_fp8, with either operand optionally given MN-major: a_mn = 1 means a_dev holds A as [Kc, M] bytes (M
 * contiguous) instead of [M, Kc]; b_mn = 1 means b_dev holds B as [Kc, Nn].  The tensor cores read such tiles
 * directly, so no transposed copy of a row-major tensor is needed to contract over its rows.  MN-major operands
 * require M to be a multiple of 256 (QE_ERR_UNSUPPORTED otherwise). */
int32_t qe_gemm_fp8_ex(const void* a_dev, uint32_t a_format, uint32_t a_mn, const void* b_dev, uint32_t b_format,
                       uint32_t b_mn, uint32_t M, uint32_t Nn, uint32_t Kc, const float* alpha_a_dev,
                       const float* alpha_b_dev, void* d_dev, uint32_t out_kind, float* amax_dev, uint32_t* status_dev,
                       void* stream);

/* Two to eight independent FP8 GEMMs in ONE kernel launch (the launch shape the layer uses for F + dI pairs and for
 * the weight gradients of a microbatch): the persistent CTAs work through the problems' tiles one problem after the
 * other, so the launch cost is paid once and partial waves are shared.  Each problem as in qe_gemm_fp8_ex; every M
 * must be a multiple of 256 (QE_ERR_UNSUPPORTED otherwise); outputs must not overlap.  descs: host array. */
typedef struct qe_gemm_desc {
  const void* a_dev;
  const void* b_dev;
  void* d_dev;
  const float* alpha_a_dev;
  const float* alpha_b_dev;
  float* amax_dev;        /* out_kind 0 only; may be NULL */
  uint32_t a_format, a_mn, b_format, b_mn;
  uint32_t M, Nn, Kc, out_kind;
} qe_gemm_desc;
int32_t qe_gemm_fp8_group(const qe_gemm_desc* descs, uint32_t n, uint32_t* status_dev, void* stream);

/* (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 * The copied-gradient step without any allocation: D = (A . B^T) * *alpha_a_dev * *alpha_b_dev is written to a
 * staging area that is built into the library (a fixed device array of qe_noalloc_staging_elems() = 2^20 FP32
 * elements, 4 MiB, resident on every GPU that loads the library until the process exits), then
 * dst_dev[i] = staging[i] (accumulate = 0) or dst_dev[i] += staging[i] (accumulate != 0).  Intended for code that
 * runs where cudaMalloc is off limits: inside another framework's allocator lock, on a thread or in a callback that
 * must not allocate, or in a process whose device memory was handed out completely at start-up.  The caller still
 * passes every input and the output; this call and everything under it call no cudaMalloc/cudaFree and no allocating
 * library routine.  A, B, shapes, formats, alphas and status_dev are as in qe_gemm_fp8; dst_dev is FP32 [M,Nn],
 * 16-byte aligned.  M*Nn above 2^20 is rejected with QE_ERR_UNSUPPORTED.  The staging area used is the CURRENT
 * device's: the current device must be the one `stream` and every pointer belong to (the call does not check it).
 * The first call on each device is a warm-up: it looks up the staging area's device address and sets kernel
 * attributes, and with lazy module loading the driver places this library's code and the 4 MiB array in device
 * memory at that point -- so make that first call where the driver may still do so (not under an allocator lock, not
 * in a fully partitioned process) and outside any stream capture.  Later calls on that device touch no allocator.
 * All calls share the one staging area and it keeps the previous call's contents: every call overwrites the part
 * it uses before reading it, so nothing needs clearing, but two calls whose work overlaps on the GPU (different
 * streams without an ordering between them) race on it -- keep them on one stream or order them with events. */
int32_t qe_gemm_fp8_staged_noalloc(const void* a_dev, uint32_t a_format, const void* b_dev, uint32_t b_format,
                                   uint32_t M, uint32_t Nn, uint32_t Kc, const float* alpha_a_dev,
                                   const float* alpha_b_dev, float* dst_dev, int32_t accumulate, uint32_t* status_dev,
                                   void* stream);
uint64_t qe_noalloc_staging_elems(void);

const char* qe_last_error(void);
const char* qe_status_name(int32_t status);
/* Version of this ABI (bumped on incompatible change). */
uint32_t qe_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QE_H_ */
