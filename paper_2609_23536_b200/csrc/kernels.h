// Kernel parameter blocks and host-side launch descriptors shared by the execution layer.
// Every kernel of the library takes exactly one by-value parameter struct, so that a launch is fully
// described by (function, grid, block, dynamic shared memory, parameter bytes) and the same description
// serves an eager launch, a CUDA-graph kernel node and a later in-place update of that node.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace qe {

// ---- device-resident layer state (lives at the start of the caller's workspace) -------------------------------
struct DevState {
  float scale[4];              // indexed by qe_tensor_class
  float scale_inv[4];
  uint32_t count[4];           // commits so far
  uint32_t pending_amax[4];    // non-negative FP32 bit patterns, accumulated with atomicMax, cleared by commit
  unsigned long long token;    // effect token as counted on the device
  float cache_sinv_W;          // inverse weight scale at the last cache refresh
  uint32_t status;             // error bits ORed in by kernels whose bounded waits expired
  float slot_sinv_X[64];       // inverse scales snapshotted when X_m / dY_m were quantised (per tape slot)
  float slot_sinv_G[64];
  uint32_t ticket;             // "last CTA" counter of the kernel whose tail performs the commit; self-resetting
  uint32_t wmax[4];            // bit pattern of max(history ring) per class, kept by the commit (derived state)
  uint32_t status_all;         // scratch of the multi-layer boundary: OR of several layers' status words
  uint32_t pad[38];            // header is 768 bytes; history rings [4][H] follow
};
static_assert(sizeof(DevState) == 768, "DevState layout");

struct CommitParams {
  DevState* st;                // null: nothing to commit
  float* hist;                 // [4][H]
  uint32_t H;
  uint32_t class_mask;         // bit c set: commit class c from pending_amax[c] (or from amax_override)
  float pow2_neg_margin;       // 2^-margin
  uint32_t bump_token;         // 1 for F and dI, 0 otherwise
  const float* amax_override;  // if non-null: value to push for the single class in class_mask
};

struct QuantParams {
  const uint16_t* x;           // bf16 [rows, cols]
  uint8_t* q;                  // fp8 [rows, cols]
  uint8_t* qT;                 // fp8 [cols, rows] or null
  uint32_t rows, cols;
  const float* scale;          // device scalar read by every thread
  const float* sinv_src;       // if non-null, block 0 copies *sinv_src to *sinv_dst (tape snapshot)
  float* sinv_dst;
  uint32_t* amax_bits;         // atomicMax target or null
  int32_t fmt;                 // 0 = E4M3, 1 = E5M2
  CommitParams commit;         // performed by the last block to finish (commit.st != null)
};


struct QuantMultiParams {
  QuantParams q[8];            // none carries a commit tail
  uint32_t block_end[8];       // cumulative block counts
  uint32_t n;
  uint32_t pad[3];
};

struct AmaxParams {
  const uint4* x;              // bf16, 8 per vector
  uint64_t nvec;
  float* partials;
  float* out;
  uint32_t nparts;
  uint32_t pad;
};

struct AccumParams {
  float4* dst;
  const float4* src;
  uint64_t nvec;
  int32_t accumulate;
  int32_t pad;
};

// Sum of M bf16 views (view m at views + m * view_vec 16-byte vectors) into FP32, added in view order.
struct ArenaReduceParams {
  const uint4* views;   // 8 bf16 per vector
  float4* dst;          // 2 vectors of 4 FP32 per input vector
  uint64_t view_vec;    // vectors per view (= N*K / 8)
  uint32_t M;
  uint32_t pad;
};

struct GemmParams {
  CUtensorMap tmA;             // A [M, Kc] bytes, box 128 x 128, 128-byte swizzle
  CUtensorMap tmB;             // B [N, Kc] bytes, box 128 x gemm_b_box_rows(M)
  CUtensorMap tmD;             // D [M, N] (bf16, FP32 or FP8 bytes), box 32 x 32, for the epilogue's bulk stores
  uint32_t M, N, Kc;
  uint32_t idesc;              // tcgen05 instruction descriptor (formats, majors, shape)
  uint32_t a_mn, b_mn;         // operand given MN-major (as [Kc, M] / [Kc, N] bytes): paired variant only
  const float* alpha_a;
  const float* alpha_b;
  void* out;                   // bf16 or FP32 [M, N], row pitch ldo elements
  uint32_t ldo;
  int32_t epi;                 // 0 bf16 (+amax), 1 FP32 overwrite, 2 FP32 accumulate, 3 FP8 hand-off (below)
  uint32_t* amax_bits;         // or null
  // epi 3: the bf16-rounded result is not stored; it is quantised for the consuming linear as that linear's own
  // cast kernel would have done: q = fp8(fp32(bf16(D)) * *out_scale), max|bf16(D)| also into *amax_bits2, and
  // *sinv_dst = *sinv_src (the consumer's tape snapshot)
  const float* out_scale;
  int32_t out_fmt;             // 0 = E4M3, 1 = E5M2
  uint32_t pad0;
  uint32_t* amax_bits2;        // or null
  const float* sinv_src;
  float* sinv_dst;
  uint32_t* status;
  CommitParams commit;         // performed by the last CTA to finish (commit.st != null)
};

// Up to eight independent GEMMs computed by one launch: tiles are numbered problem after problem.
struct GemmGroupParams {
  uint32_t n;
  uint32_t tile_end[8];        // cumulative tile counts (256 x 256 tiles)
  uint32_t pad[7];
  GemmParams prob[8];
};

// ORs the status words of up to 64 layers into *out (first chunk: out = OR; later chunks: out |= OR).
struct StatusGatherParams {
  const uint32_t* src[64];
  uint32_t* out;
  uint32_t n;
  uint32_t accumulate;
};

// One launch, self-contained.
struct Launch {
  const void* func = nullptr;
  dim3 grid{1, 1, 1}, block{1, 1, 1};
  uint32_t smem = 0;
  uint32_t nbytes = 0;
  alignas(64) unsigned char params[4864];
  template <class P>
  void set(const P& p) {
    static_assert(sizeof(P) <= sizeof(params), "parameter block too large");
    nbytes = sizeof(P);
    __builtin_memcpy(params, &p, sizeof(P));
  }
};

Launch make_quantize(const QuantParams& p);
Launch make_quantize_multi(const QuantParams* casts, uint32_t n);  // 2..8 independent casts in one launch
Launch make_commit(const CommitParams& p);
Launch make_status_gather(const StatusGatherParams& p);
Launch make_amax_pass1(const AmaxParams& p);
Launch make_amax_pass2(const AmaxParams& p);
Launch make_accumulate(const AccumParams& p);
Launch make_arena_reduce(const ArenaReduceParams& p);
Launch make_gemm(const GemmParams& p, int num_sms);
// One launch for n = 2..8 GEMMs (each may carry its own commit tail); false if the group cannot be formed (a problem
// needs the single-CTA variant), in which case the caller launches them one by one.
bool make_gemm_group(const GemmParams* probs, uint32_t n, int num_sms, Launch* out);
cudaError_t gemm_prepare();  // opt in to the dynamic shared memory the GEMM needs (once per device)
uint32_t gemm_idesc(int a_fmt, int b_fmt, uint32_t M, bool a_mn = false, bool b_mn = false);
bool gemm_uses_pair(uint32_t M);
uint32_t gemm_b_box_rows(uint32_t M);  // rows of the B operand's TMA box for a GEMM with M rows (128 paired, 256 single)
constexpr uint32_t kAmaxPartials = 2048;

}  // namespace qe
