// Amax-history reduction and scale update as a device function, shared by the standalone commit kernel and by the
// tails of the quantise and GEMM kernels (where the last block to finish performs it, saving a launch).
//   hist[c][count mod H] = amax;  scale_c = fp8_max / max(hist[c]) / 2^margin;  scale_inv_c = 1 / scale_c
// 256 threads take part: 64 per tensor class, all four classes in parallel, one barrier.  The ring's maximum is kept
// beside it so that a commit usually reads one entry instead of H.  The maximum is taken on
// the bit patterns of the non-negative FP32 entries, which orders them like their values and lets a NaN or Inf
// entry surface as "not finite" (scale then stays as it was, like for an all-zero window).
#pragma once
#include <cfloat>

#include "kernels.h"

namespace qe {

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic stream serialization, so
// the next kernel in the stream may be scheduled while this one drains.  grid_dep_wait() returns once every kernel
// this one depends on has completed and its writes are visible: it must precede the first access to anything a
// predecessor produced.  grid_dep_launch() lets the successor's blocks start (they stop at their own wait).
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <class Sync>
__device__ __forceinline__ void commit_classes(const CommitParams& p, int tid, uint32_t* red /* shared, 8 words */,
                                               Sync sync) {
  DevState* st = p.st;
  const int c = tid >> 6, g = tid & 63;
  const bool active = (p.class_mask >> c) & 1u;
  uint32_t m = 0, newest = 0, cnt = 0, pos = 0;
  uint32_t* h = reinterpret_cast<uint32_t*>(p.hist + (size_t)c * p.H);
  if (active) {
    cnt = __ldcg(&st->count[c]);
    newest = p.amax_override ? (__float_as_uint(__ldcg(p.amax_override)) & 0x7fffffffu) : __ldcg(&st->pending_amax[c]);
    const uint32_t wmax = __ldcg(&st->wmax[c]);  // maximum of the ring as it stands
    pos = cnt % p.H;
    const uint32_t evicted = __ldcg(h + pos);
    // The new maximum is known without reading the ring unless the entry that leaves was the maximum and the one
    // that enters is smaller: only then is the ring scanned (exactly the same value either way).
    if (newest >= wmax) m = newest;
    else if (evicted < wmax) m = wmax;
    else
      for (uint32_t i = g; i < p.H; i += 64) m = max(m, i == pos ? newest : __ldcg(h + i));
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  sync();
  if (active && g == 0) {
    m = max(red[2 * c], red[2 * c + 1]);
    h[pos] = newest;
    st->count[c] = cnt + 1;
    st->pending_amax[c] = 0;
    st->wmax[c] = m;
    if (m != 0 && m < 0x7f800000u) {
      const float fp8_max = c == 2 ? 57344.0f : 448.0f;  // class 2 = gradients (E5M2), others E4M3
      float s = __fmul_rn(__fdiv_rn(fp8_max, __uint_as_float(m)), p.pow2_neg_margin);
      if (isinf(s)) s = FLT_MAX;
      st->scale[c] = s;
      st->scale_inv[c] = __fdiv_rn(1.0f, s);
    }
  }
  if (tid == 0 && p.bump_token) st->token += 1ull;
}

// The same commit done by ONE warp: eight lanes per tensor class (the rare ring scan strides by eight).  A grouped GEMM
// launch ends with up to eight commits, one per problem; its last CTA gives each of them to an epilogue warp of its
// own instead of running them one after the other (each is a chain of dependent global accesses, ~1.5 us: at launches
// of 20 us that was half the launch).  Same values as commit_classes; the token is bumped atomically because two
// problems of one launch may belong to the same layer (its forward and its input gradient of different microbatches).
__device__ __forceinline__ void commit_classes_warp(const CommitParams& p, int lane) {
  DevState* st = p.st;
  const int c = lane >> 3, g = lane & 7;
  const bool active = (p.class_mask >> c) & 1u;
  uint32_t m = 0, newest = 0, cnt = 0, pos = 0;
  uint32_t* h = reinterpret_cast<uint32_t*>(p.hist + (size_t)c * p.H);
  if (active) {
    cnt = __ldcg(&st->count[c]);
    newest = p.amax_override ? (__float_as_uint(__ldcg(p.amax_override)) & 0x7fffffffu) : __ldcg(&st->pending_amax[c]);
    const uint32_t wmax = __ldcg(&st->wmax[c]);
    pos = cnt % p.H;
    const uint32_t evicted = __ldcg(h + pos);
    if (newest >= wmax) m = newest;
    else if (evicted < wmax) m = wmax;
    else
      for (uint32_t i = g; i < p.H; i += 8) m = max(m, i == pos ? newest : __ldcg(h + i));
  }
  m = max(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = max(m, __shfl_xor_sync(0xffffffffu, m, 2));
  m = max(m, __shfl_xor_sync(0xffffffffu, m, 4));
  if (active && g == 0) {
    h[pos] = newest;
    st->count[c] = cnt + 1;
    st->pending_amax[c] = 0;
    st->wmax[c] = m;
    if (m != 0 && m < 0x7f800000u) {
      const float fp8_max = c == 2 ? 57344.0f : 448.0f;
      float s = __fmul_rn(__fdiv_rn(fp8_max, __uint_as_float(m)), p.pow2_neg_margin);
      if (isinf(s)) s = FLT_MAX;
      st->scale[c] = s;
      st->scale_inv[c] = __fdiv_rn(1.0f, s);
    }
  }
  if (lane == 0 && p.bump_token) atomicAdd(&st->token, 1ull);
}

// Returns true in every thread of exactly one block of the grid: the last one to get here.  Stores and atomics the
// grid made before this call are visible to that block afterwards.
template <class Sync>
__device__ __forceinline__ bool last_block(uint32_t* ticket, uint32_t nblocks, int tid, uint32_t* flag /* shared */,
                                           Sync sync) {
  __threadfence();
  sync();
  if (tid == 0) {
    const uint32_t t = atomicAdd(ticket, 1u);
    const bool last = t == nblocks - 1;
    if (last) atomicExch(ticket, 0u);  // ready for the next kernel that uses it
    *flag = last ? 1u : 0u;
  }
  sync();
  const bool last = *flag != 0u;
  if (last) __threadfence();
  return last;
}

}  // namespace qe
