// Bandwidth-bound kernels of the path: fused cast-to-FP8 with amax and transposed copy, the amax-history /
// scale update, a standalone two-pass amax, and the FP32 copy-add of the copied-gradient comparison path.
// Written for sm_100a: 16-byte loads, 8-byte stores that always fill whole 32-byte sectors, no shared-memory
// staging (the 8x8 byte transpose is done in registers), warp-shuffle reductions.
#include <cuda_fp8.h>

#include <cfloat>

#include "commit.cuh"
#include "kernels.h"

namespace qe {

// ------------------------------------------------------------------------------------------------ helpers
__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) { return __reduce_max_sync(0xffffffffu, v); }

// Largest magnitude pattern of the 8 bf16 values in a 16-byte vector (as two packed 15-bit magnitudes).
__device__ __forceinline__ uint32_t absmax_packed(uint32_t m, const uint4& v) {
  m = __vmaxu2(m, v.x & 0x7fff7fffu);
  m = __vmaxu2(m, v.y & 0x7fff7fffu);
  m = __vmaxu2(m, v.z & 0x7fff7fffu);
  m = __vmaxu2(m, v.w & 0x7fff7fffu);
  return m;
}
// packed pair of bf16 magnitudes -> FP32 bit pattern of the larger
__device__ __forceinline__ uint32_t packed_to_f32bits(uint32_t m) { return max(m & 0xffffu, m >> 16) << 16; }

template <int FMT>
__device__ __forceinline__ uint32_t cast4(uint32_t w0, uint32_t w1, float scale) {
  // w0 = {x0 (low half), x1}, w1 = {x2, x3} as bf16; product rounded to FP32 once, then RNE + saturate to FP8
  const float f0 = __fmul_rn(__uint_as_float(w0 << 16), scale);
  const float f1 = __fmul_rn(__uint_as_float(w0 & 0xffff0000u), scale);
  const float f2 = __fmul_rn(__uint_as_float(w1 << 16), scale);
  const float f3 = __fmul_rn(__uint_as_float(w1 & 0xffff0000u), scale);
  constexpr __nv_fp8_interpretation_t kind = FMT == 0 ? __NV_E4M3 : __NV_E5M2;
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(f0, f1), __NV_SATFINITE, kind);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(f2, f3), __NV_SATFINITE, kind);
  return lo | (hi << 16);
}

// 4x4 byte transpose: a[i] holds row i (byte j = column j); t[j] receives column j (byte i = row i).
__device__ __forceinline__ void transpose4x4(const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                             const uint32_t a3, uint32_t* t) {
  const uint32_t p0 = __byte_perm(a0, a1, 0x5140), p1 = __byte_perm(a2, a3, 0x5140);
  const uint32_t p2 = __byte_perm(a0, a1, 0x7362), p3 = __byte_perm(a2, a3, 0x7362);
  t[0] = __byte_perm(p0, p1, 0x5410);
  t[1] = __byte_perm(p0, p1, 0x7632);
  t[2] = __byte_perm(p2, p3, 0x5410);
  t[3] = __byte_perm(p2, p3, 0x7632);
}

// ------------------------------------------------------------------------------------------------ quantise
// Block = 8 warps stacked along rows, covering 256 rows x 64 columns.  A warp covers 32 rows x 64 columns as
// 4 x 8 threads, each owning an 8 x 8 element block: eight 16-byte loads (a warp instruction reads four full
// 128-byte row segments), eight 8-byte row-major stores (four 64-byte segments per instruction) and eight 8-byte
// transposed stores (per instruction eight full 32-byte sectors; the block's eight warps complete 256 contiguous
// bytes of every output row of the transposed copy).
constexpr int kQuantThreads = 256;

// One block's share (256 rows x 64 columns at block coordinates bx, by) of a cast; wmax: 8 shared words.
template <int FMT>
__device__ __forceinline__ void quantize_block(const QuantParams& p, uint32_t bx, uint32_t by, uint32_t* wmax) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rb = lane >> 3, cv = lane & 7;
  const uint32_t row0 = by * 256u + warp * 32u + rb * 8u;
  const uint32_t col0 = bx * 64u + cv * 8u;
  const float scale = *p.scale;
  if (bx == 0 && by == 0 && threadIdx.x == 0 && p.sinv_dst) *p.sinv_dst = *p.sinv_src;

  uint32_t m = 0;
  if (row0 < p.rows) {  // warp-uniform up to rb; rows is a multiple of 8 so a thread's 8 rows are all in or out
    uint4 v[8];
    const uint16_t* src = p.x + (size_t)row0 * p.cols + col0;
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldcs(reinterpret_cast<const uint4*>(src + (size_t)i * p.cols));
    uint32_t lo[8], hi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      m = absmax_packed(m, v[i]);
      lo[i] = cast4<FMT>(v[i].x, v[i].y, scale);
      hi[i] = cast4<FMT>(v[i].z, v[i].w, scale);
    }
    uint8_t* dst = p.q + (size_t)row0 * p.cols + col0;
#pragma unroll
    for (int i = 0; i < 8; ++i) *reinterpret_cast<uint2*>(dst + (size_t)i * p.cols) = make_uint2(lo[i], hi[i]);
    if (p.qT) {
      uint32_t t00[4], t10[4], t01[4], t11[4];  // t<rowhalf><colhalf>
      transpose4x4(lo[0], lo[1], lo[2], lo[3], t00);
      transpose4x4(lo[4], lo[5], lo[6], lo[7], t10);
      transpose4x4(hi[0], hi[1], hi[2], hi[3], t01);
      transpose4x4(hi[4], hi[5], hi[6], hi[7], t11);
      uint8_t* dT = p.qT + (size_t)col0 * p.rows + row0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        *reinterpret_cast<uint2*>(dT + (size_t)j * p.rows) = make_uint2(t00[j], t10[j]);
        *reinterpret_cast<uint2*>(dT + (size_t)(j + 4) * p.rows) = make_uint2(t01[j], t11[j]);
      }
    }
  }
  if (p.amax_bits) {
    const uint32_t w = warp_max_u32(packed_to_f32bits(m));
    if (lane == 0) wmax[warp] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t b = wmax[0];
#pragma unroll
      for (int i = 1; i < kQuantThreads / 32; ++i) b = max(b, wmax[i]);
      if (b) atomicMax(p.amax_bits, b);
    }
  }
}

template <int FMT>
__global__ void __launch_bounds__(kQuantThreads) quantize_kernel(const __grid_constant__ QuantParams p) {
  __shared__ uint32_t wmax[kQuantThreads / 32];
  __shared__ uint32_t last_flag;
  grid_dep_wait();  // the scale (and possibly x) come from earlier kernels
  grid_dep_launch();
  quantize_block<FMT>(p, blockIdx.x, blockIdx.y, wmax);
  if (p.commit.st) {  // the last block to finish folds the new amax into the history and updates the scale
    auto sync = [] { __syncthreads(); };
    if (last_block(&p.commit.st->ticket, gridDim.x * gridDim.y, threadIdx.x, &last_flag, sync))
      commit_classes(p.commit, threadIdx.x, wmax, sync);
  }
}

// Two to eight independent casts in one launch (the X of forward units and the dY of input-gradient units that go out
// together): the blocks are dealt to the casts one cast after the other.  No commit tails.
__global__ void __launch_bounds__(kQuantThreads) quantize_multi_kernel(const __grid_constant__ QuantMultiParams mp) {
  __shared__ uint32_t wmax[kQuantThreads / 32];
  grid_dep_wait();
  grid_dep_launch();
  uint32_t which = 0, base = 0;
  while (which + 1 < mp.n && blockIdx.x >= mp.block_end[which]) base = mp.block_end[which++];
  const QuantParams& p = mp.q[which];
  const uint32_t b = blockIdx.x - base, bxn = p.cols / 64u;
  if (p.fmt == 0) quantize_block<0>(p, b % bxn, b / bxn, wmax);
  else quantize_block<1>(p, b % bxn, b / bxn, wmax);
}

Launch make_quantize_multi(const QuantParams* casts, uint32_t n) {
  QuantMultiParams mp{};
  uint32_t blocks = 0;
  for (uint32_t i = 0; i < n; ++i) {
    mp.q[i] = casts[i];
    blocks += (casts[i].cols / 64) * ((casts[i].rows + 255) / 256);
    mp.block_end[i] = blocks;
  }
  mp.n = n;
  Launch l;
  l.func = (const void*)quantize_multi_kernel;
  l.grid = dim3(blocks, 1, 1);
  l.block = dim3(kQuantThreads, 1, 1);
  l.set(mp);
  return l;
}

Launch make_quantize(const QuantParams& p) {
  Launch l;
  l.func = p.fmt == 0 ? (const void*)quantize_kernel<0> : (const void*)quantize_kernel<1>;
  l.grid = dim3(p.cols / 64, (p.rows + 255) / 256, 1);
  l.block = dim3(kQuantThreads, 1, 1);
  l.set(p);
  return l;
}

// ------------------------------------------------------------------------------------------------ commit
// The scale update as a kernel of its own (one block; latency-bound: at most 16 KB read).
__global__ void __launch_bounds__(256) commit_kernel(const __grid_constant__ CommitParams p) {
  __shared__ uint32_t red[8];
  grid_dep_wait();
  grid_dep_launch();
  commit_classes(p, threadIdx.x, red, [] { __syncthreads(); });
}

__global__ void __launch_bounds__(64) status_gather_kernel(const __grid_constant__ StatusGatherParams p) {
  grid_dep_wait();
  grid_dep_launch();
  uint32_t v = threadIdx.x < p.n ? __ldcg(p.src[threadIdx.x]) : 0u;
  v = __reduce_or_sync(0xffffffffu, v);
  __shared__ uint32_t w[2];
  if ((threadIdx.x & 31) == 0) w[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) *p.out = (p.accumulate ? *p.out : 0u) | w[0] | w[1];
}

Launch make_status_gather(const StatusGatherParams& p) {
  Launch l;
  l.func = (const void*)status_gather_kernel;
  l.grid = dim3(1, 1, 1);
  l.block = dim3(64, 1, 1);
  l.set(p);
  return l;
}

Launch make_commit(const CommitParams& p) {
  Launch l;
  l.func = (const void*)commit_kernel;
  l.block = dim3(256, 1, 1);
  l.set(p);
  return l;
}

// ------------------------------------------------------------------------------------------------ standalone amax
__global__ void __launch_bounds__(256) amax_pass1_kernel(const __grid_constant__ AmaxParams p) {
  __shared__ uint32_t wmax[8];
  uint32_t m = 0;
  grid_dep_wait();
  grid_dep_launch();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // four independent 16-byte loads in flight per thread
  for (; i + 3 * stride < p.nvec; i += 4 * stride) {
    const uint4 a = __ldcs(p.x + i), b = __ldcs(p.x + i + stride), c = __ldcs(p.x + i + 2 * stride),
                d = __ldcs(p.x + i + 3 * stride);
    m = absmax_packed(absmax_packed(absmax_packed(absmax_packed(m, a), b), c), d);
  }
  for (; i < p.nvec; i += stride) m = absmax_packed(m, __ldcs(p.x + i));
  const uint32_t w = warp_max_u32(packed_to_f32bits(m));
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = w;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t b = wmax[0];
    for (int k = 1; k < 8; ++k) b = max(b, wmax[k]);
    p.partials[blockIdx.x] = __uint_as_float(b);
  }
}

__global__ void __launch_bounds__(256) amax_pass2_kernel(const __grid_constant__ AmaxParams p) {
  __shared__ uint32_t wmax[8];
  uint32_t m = 0;
  grid_dep_wait();
  grid_dep_launch();
  for (uint32_t i = threadIdx.x; i < p.nparts; i += blockDim.x) m = max(m, __float_as_uint(p.partials[i]));
  m = warp_max_u32(m);
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < 8; ++k) m = max(m, wmax[k]);
    *p.out = __uint_as_float(m);
  }
}

Launch make_amax_pass1(const AmaxParams& p) {
  Launch l;
  l.func = (const void*)amax_pass1_kernel;
  l.grid = dim3(p.nparts, 1, 1);
  l.block = dim3(256, 1, 1);
  l.set(p);
  return l;
}
Launch make_amax_pass2(const AmaxParams& p) {
  Launch l;
  l.func = (const void*)amax_pass2_kernel;
  l.block = dim3(256, 1, 1);
  l.set(p);
  return l;
}

// ------------------------------------------------------------------------------------------------ copy-add
__global__ void __launch_bounds__(256) accumulate_kernel(const __grid_constant__ AccumParams p) {
  grid_dep_wait();
  grid_dep_launch();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < p.nvec; i += stride) {
    float4 s = __ldcs(p.src + i);
    if (p.accumulate) {
      const float4 d = p.dst[i];
      s.x = __fadd_rn(d.x, s.x);
      s.y = __fadd_rn(d.y, s.y);
      s.z = __fadd_rn(d.z, s.z);
      s.w = __fadd_rn(d.w, s.w);
    }
    p.dst[i] = s;
  }
}

Launch make_accumulate(const AccumParams& p) {
  Launch l;
  l.func = (const void*)accumulate_kernel;
  const uint64_t blocks = (p.nvec + 255) / 256;
  l.grid = dim3((unsigned)(blocks < 148ull * 16 ? (blocks ? blocks : 1) : 148ull * 16), 1, 1);
  l.block = dim3(256, 1, 1);
  l.set(p);
  return l;
}

// ------------------------------------------------------------------------------------------------ arena reduction
// The per-microbatch arena (one bf16 view per matrix parameter and microbatch): the optimizer-visible FP32 gradient
// is the sum of the M views, added in microbatch order.  (2 M + 4) bytes per element; a thread owns 8 consecutive
// elements, the loads of four views are in flight at once.
__device__ __forceinline__ void add_bf16x8(float (&a)[8], const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    a[2 * j] = __fadd_rn(a[2 * j], __uint_as_float(w[j] << 16));
    a[2 * j + 1] = __fadd_rn(a[2 * j + 1], __uint_as_float(w[j] & 0xffff0000u));
  }
}

__global__ void __launch_bounds__(256) arena_reduce_kernel(const __grid_constant__ ArenaReduceParams p) {
  grid_dep_wait();
  grid_dep_launch();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < p.view_vec; i += stride) {
    const uint4* src = p.views + i;
    const uint4 v0 = __ldcs(src);
    const uint32_t w[4] = {v0.x, v0.y, v0.z, v0.w};
    float a[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      a[2 * j] = __uint_as_float(w[j] << 16);
      a[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
    uint32_t m = 1;
    for (; m + 4 <= p.M; m += 4) {
      const uint4 x0 = __ldcs(src + (uint64_t)m * p.view_vec), x1 = __ldcs(src + (uint64_t)(m + 1) * p.view_vec);
      const uint4 x2 = __ldcs(src + (uint64_t)(m + 2) * p.view_vec), x3 = __ldcs(src + (uint64_t)(m + 3) * p.view_vec);
      add_bf16x8(a, x0);
      add_bf16x8(a, x1);
      add_bf16x8(a, x2);
      add_bf16x8(a, x3);
    }
    for (; m < p.M; ++m) add_bf16x8(a, __ldcs(src + (uint64_t)m * p.view_vec));
    p.dst[2 * i] = make_float4(a[0], a[1], a[2], a[3]);
    p.dst[2 * i + 1] = make_float4(a[4], a[5], a[6], a[7]);
  }
}

Launch make_arena_reduce(const ArenaReduceParams& p) {
  Launch l;
  l.func = (const void*)arena_reduce_kernel;
  const uint64_t blocks = (p.view_vec + 255) / 256;
  l.grid = dim3((unsigned)(blocks < 148ull * 8 ? (blocks ? blocks : 1) : 148ull * 8), 1, 1);
  l.block = dim3(256, 1, 1);
  l.set(p);
  return l;
}

}  // namespace qe
