// The kernels of the path as standalone calls (no layer state): casts, amax, copy-add, arena reduction, FP8 GEMMs.
#include "layer_impl.h"

using namespace qe_impl;

extern "C" {

// ------------------------------------------------------------------------------------------------ standalone kernels
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
