// Tracker, advantage and sampling kernels: the small group-free pieces of SPO.
// All are memory-streaming kernels: coalesced vector loads of the interleaved
// (alpha, beta) table, warp-shuffle reductions, integer prefix sums.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include <mutex>

#include "spo_internal.h"

namespace spo {

namespace {

__device__ __forceinline__ void flag(int32_t* d_status, int bit) {
  if (d_status) atomicOr(d_status, bit);
}

// ---------------------------------------------------------------------------
// Algorithm 2: alpha0 = N0*v0, beta0 = N0*(1-v0)
// ---------------------------------------------------------------------------
__global__ void tracker_init_kernel(float2* __restrict__ ab, const float* __restrict__ v0, int64_t N, float n0) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < N; i += stride) {
    float v = v0[i];
    ab[i] = make_float2(n0 * v, n0 * (1.0f - v));
  }
}

// ---------------------------------------------------------------------------
// Sampling weight of one table entry (Eq. "sampling_coef"), w = sqrt(v(1-v)) + eps with
// v(1-v) = alpha beta / (alpha+beta)^2, in fp32 as a fixed sequence of individually rounded
// operations (no contraction into FMAs) so that a host restatement gives the same bits:
//   n = a+b; t = a*b; den = n*n; x = t*den;
//   common case, 2^-100 <= x <= 2^100 and a > 0:  s = t * y  with y ~ 1/sqrt(x) = 1/(sqrt(t) n):
//     y0 = bits(0x5f3759df - (bits(x) >> 1)); three Newton steps y <- y*(1.5 - (0.5x)*(y*y));
//   n == 0 (empty entry): s = 0.5;   a or b zero (n > 0): s = 0;
//   any other magnitude: s = sqrt((a/n)*(b/n)) with IEEE division and square root;
//   w = s + eps.
// The Newton form needs 20 plain multiplies / subtracts where a correctly rounded reciprocal and
// square root need about twice that; the table scan is bound by instruction issue, so this is what
// sets its speed.  s is within 3e-7 relative of the exact value.
// A negative or non-finite entry yields weight 0 and sets SPO_DEV_NONFINITE in *d_status.
// ---------------------------------------------------------------------------
// Everything but the common case, out of line so that the scan's hot loop stays short:
// invalid entries (weight 0, status bit), empty entries, a zero alpha or beta, extreme magnitudes.
__device__ __noinline__ float entry_weight_uncommon(float a, float b, float eps, int32_t* d_status) {
  const float n = __fadd_rn(a, b);
  if ((fminf(a, b) < 0.0f) | !(n < CUDART_INF_F)) {                  // negative, NaN or Inf
    flag(d_status, SPO_DEV_NONFINITE);
    return 0.0f;
  }
  float s;
  if (n == 0.0f) s = 0.5f;
  else if (fminf(a, b) == 0.0f) s = 0.0f;
  else s = __fsqrt_rn(__fmul_rn(__fdiv_rn(a, n), __fdiv_rn(b, n)));
  return __fadd_rn(s, eps);
}

__device__ __forceinline__ float entry_weight(float a, float b, float eps, int32_t* d_status) {
  const float n = __fadd_rn(a, b);
  const float t = __fmul_rn(a, b);
  const float x = __fmul_rn(t, __fmul_rn(n, n));
  // x in range and a > 0 imply b > 0 and everything finite: one test covers validity too
  if (!((x >= 0x1p-100f) & (x <= 0x1p100f) & (a > 0.0f))) return entry_weight_uncommon(a, b, eps, d_status);
  const float h = __fmul_rn(0.5f, x);
  float y = __uint_as_float(0x5f3759dfu - (__float_as_uint(x) >> 1));
#pragma unroll
  for (int k = 0; k < 3; ++k) y = __fmul_rn(y, __fsub_rn(1.5f, __fmul_rn(h, __fmul_rn(y, y))));
  return __fadd_rn(__fmul_rn(t, y), eps);
}

// q = floor(w * 2^32): exact, the scale is a power of two (w is finite, non-negative, far below 2^32).
__device__ __forceinline__ unsigned long long quantise(float w) {
  return __float2ull_rz(w * 4294967296.0f);
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ unsigned long long warp_incl_scan_u64(unsigned long long v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned long long t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// One block = one tile of kSampleTile entries: 256 threads x 4 float4 loads (2 entries each).
// EMIT: also write the weights.  Full tiles take a path without per-load bounds tests.
template <bool EMIT>
__global__ void __launch_bounds__(256)
sample_tile_sums_kernel(const float4* __restrict__ ab4, int64_t N, float eps, float2* __restrict__ out_w2,
                        float* __restrict__ out_w, unsigned long long* __restrict__ tile_sums,
                        unsigned long long* __restrict__ super_sums, int32_t* d_status) {
  const int64_t tile = blockIdx.x;
  const int64_t first_pair = tile * (kSampleTile / 2);
  const int64_t n_pairs = N >> 1;
  unsigned long long sum = 0;
  if (first_pair + kSampleTile / 2 <= n_pairs) {
    float4 e[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) e[j] = __ldg(ab4 + first_pair + j * 256 + threadIdx.x);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float w0 = entry_weight(e[j].x, e[j].y, eps, d_status);
      const float w1 = entry_weight(e[j].z, e[j].w, eps, d_status);
      sum += quantise(w0) + quantise(w1);
      if (EMIT) out_w2[first_pair + j * 256 + threadIdx.x] = make_float2(w0, w1);
    }
  } else {
#pragma unroll 1
    for (int j = 0; j < 4; ++j) {
      const int64_t p = first_pair + j * 256 + threadIdx.x;
      if (p < n_pairs) {
        const float4 e = __ldg(ab4 + p);
        const float w0 = entry_weight(e.x, e.y, eps, d_status);
        const float w1 = entry_weight(e.z, e.w, eps, d_status);
        sum += quantise(w0) + quantise(w1);
        if (EMIT) out_w2[p] = make_float2(w0, w1);
      } else if (p == n_pairs && (N & 1)) {      // odd tail entry
        const float* ab = reinterpret_cast<const float*>(ab4);
        const float w0 = entry_weight(ab[2 * (N - 1)], ab[2 * (N - 1) + 1], eps, d_status);
        sum += quantise(w0);
        if (EMIT) out_w[N - 1] = w0;
      }
    }
  }
  sum = warp_sum_u64(sum);
  __shared__ unsigned long long s_part[8];
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += s_part[w];
    tile_sums[tile] = t;
    atomicAdd(&super_sums[tile / kSuperTile], t);      // integer adds commute: exact in any order
  }
}

// Warp-wide search of the first entry whose running sum exceeds t: `get(i)` yields entry i of a
// list of `count` non-negative integers, `run` is the sum of everything before the list.  Returns
// the index (or -1) and leaves in `run` the sum of everything before that index.
template <typename Get>
__device__ __forceinline__ int64_t warp_find(int64_t count, unsigned long long t, unsigned long long& run, int lane,
                                             Get get) {
  for (int64_t c0 = 0; c0 < count; c0 += 32) {
    const int64_t i = c0 + lane;
    const unsigned long long q = i < count ? get(i) : 0ull;
    const unsigned long long incl = warp_incl_scan_u64(q, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, run + incl > t);
    if (hit) {
      const int first = __ffs(hit) - 1;
      const unsigned long long before = __shfl_sync(0xffffffffu, incl - q, first);
      run += before;
      return c0 + first;
    }
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  return -1;
}

__device__ __forceinline__ uint32_t hash_id(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

// One warp per uniform: total weight, threshold, then three levels of search (super-tile, tile,
// entry).  The winner is also entered into an open-addressing table keyed by prompt id + 1
// (0 = empty) whose value keeps the largest M - k, i.e. the earliest draw k of that prompt.
__global__ void __launch_bounds__(256)
sample_search_kernel(const float* __restrict__ ab, int64_t N, float eps, const float* __restrict__ uniforms,
                     int32_t M, const unsigned long long* __restrict__ tile_sums,
                     const unsigned long long* __restrict__ super_sums, int64_t n_tiles, int n_super,
                     int32_t* __restrict__ cand, int32_t* __restrict__ slot_of, int32_t* keys, int32_t* vals,
                     uint32_t slot_mask, int32_t* d_status) {
  const int lane = threadIdx.x & 31;
  const int k = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (k >= M) return;
  unsigned long long wtot = 0;
  for (int i = lane; i < n_super; i += 32) wtot += super_sums[i];
  wtot = warp_sum_u64(wtot);
  const float u = uniforms[k];
  if (wtot == 0 || !(u >= 0.0f) || !(u < 1.0f)) {
    if (lane == 0) {
      cand[k] = -1;
      if (wtot != 0) flag(d_status, SPO_DEV_NONFINITE);
      else if (k == 0) flag(d_status, SPO_DEV_ZERO_TOTAL_WEIGHT);
    }
    return;
  }
  const unsigned long long bigu = __float2ull_rz(u * 4294967296.0f);          // floor(u * 2^32), exact
  const unsigned long long t = (__umul64hi(bigu, wtot) << 32) | ((bigu * wtot) >> 32);
  unsigned long long run = 0;
  int64_t off = -1, base = 0;
  const int64_t sup = warp_find(n_super, t, run, lane, [&](int64_t i) { return super_sums[i]; });
  if (sup >= 0) {                                                    // warp-uniform
    const int64_t tile0 = sup * kSuperTile;
    const int64_t tiles_here = n_tiles - tile0 < kSuperTile ? n_tiles - tile0 : kSuperTile;
    const int64_t tl = warp_find(tiles_here, t, run, lane, [&](int64_t i) { return tile_sums[tile0 + i]; });
    if (tl >= 0) {
      base = (tile0 + tl) * kSampleTile;
      const int64_t n_here = N - base < kSampleTile ? N - base : kSampleTile;
      // entries: 128 per step, four consecutive ones per lane (two float4 loads)
      const float4* ab4 = reinterpret_cast<const float4*>(ab) + base / 2;      // base is a multiple of 2048
      for (int64_t c0 = 0; c0 < n_here && off < 0; c0 += 128) {
        const int64_t i0 = c0 + 4 * lane;
        unsigned long long q[4] = {0ull, 0ull, 0ull, 0ull};
        if (i0 + 3 < n_here) {
          const float4 e0 = __ldg(ab4 + i0 / 2), e1 = __ldg(ab4 + i0 / 2 + 1);
          q[0] = quantise(entry_weight(e0.x, e0.y, eps, d_status));
          q[1] = quantise(entry_weight(e0.z, e0.w, eps, d_status));
          q[2] = quantise(entry_weight(e1.x, e1.y, eps, d_status));
          q[3] = quantise(entry_weight(e1.z, e1.w, eps, d_status));
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (i0 + j < n_here) q[j] = quantise(entry_weight(ab[2 * (base + i0 + j)], ab[2 * (base + i0 + j) + 1], eps, d_status));
        }
        const unsigned long long mine = q[0] + q[1] + q[2] + q[3];
        const unsigned long long incl = warp_incl_scan_u64(mine, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, run + incl > t);
        if (hit) {
          const int first = __ffs(hit) - 1;                              // lane whose four entries hold the answer
          unsigned long long r0 = run + __shfl_sync(0xffffffffu, incl - mine, first);
          const unsigned long long f0 = __shfl_sync(0xffffffffu, q[0], first), f1 = __shfl_sync(0xffffffffu, q[1], first),
                                   f2 = __shfl_sync(0xffffffffu, q[2], first);
          int j = 3;
          if (r0 + f0 > t) j = 0;
          else if (r0 + f0 + f1 > t) j = 1;
          else if (r0 + f0 + f1 + f2 > t) j = 2;
          off = c0 + 4 * first + j;
        } else {
          run += __shfl_sync(0xffffffffu, incl, 31);
        }
      }
    }
  }
  if (lane == 0) {
    const int32_t found = off < 0 ? -1 : (int32_t)(base + off);
    cand[k] = found;
    if (found >= 0) {
      uint32_t s = hash_id((uint32_t)found) & slot_mask;
      for (uint32_t probe = 0; probe <= slot_mask; ++probe) {
        const int32_t prev = atomicCAS(&keys[s], 0, found + 1);
        if (prev == 0 || prev == found + 1) { atomicMax(&vals[s], M - k); slot_of[k] = (int32_t)s; break; }
        s = (s + 1) & slot_mask;
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Small tables (N <= kSmallTableMax): the same draw, organised for latency.
// ---------------------------------------------------------------------------
// The four kernels of this path are a few microseconds each, so the gaps between them count.  Each one
// lets the next be set up while it still runs (programmatic dependent launch): pdl_release() at the top
// of a kernel allows its successor's blocks onto the SMs, pdl_wait() at the top of the successor holds them
// until the predecessor has finished and its writes are visible.  Every kernel of the chain waits before
// it touches anything a predecessor writes, so completion of one implies completion of all before it.
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// One block = one tile of kSmallTile entries: 128 threads, one float4 (two entries) each.
template <bool EMIT>
__global__ void __launch_bounds__(kSmallTile / 2)
sample_small_sums_kernel(const float4* __restrict__ ab4, int64_t N, float eps, float2* __restrict__ out_w2,
                         float* __restrict__ out_w, unsigned long long* __restrict__ tile_sums,
                         int32_t* __restrict__ first_draw, int32_t* d_status) {
  pdl_release();
  const int64_t p = (int64_t)blockIdx.x * (kSmallTile / 2) + threadIdx.x;
  const int64_t n_pairs = N >> 1;
  unsigned long long sum = 0;
  // first_draw[id] will hold the largest M - k over the draws k that pick prompt id: cleared here
  if (p < n_pairs) reinterpret_cast<int2*>(first_draw)[p] = make_int2(0, 0);
  else if (p == n_pairs && (N & 1)) first_draw[N - 1] = 0;
  if (p < n_pairs) {
    const float4 e = __ldg(ab4 + p);
    const float w0 = entry_weight(e.x, e.y, eps, d_status);
    const float w1 = entry_weight(e.z, e.w, eps, d_status);
    sum = quantise(w0) + quantise(w1);
    if (EMIT) out_w2[p] = make_float2(w0, w1);
  } else if (p == n_pairs && (N & 1)) {          // odd tail entry
    const float* ab = reinterpret_cast<const float*>(ab4);
    const float w0 = entry_weight(ab[2 * (N - 1)], ab[2 * (N - 1) + 1], eps, d_status);
    sum = quantise(w0);
    if (EMIT) out_w[N - 1] = w0;
  }
  sum = warp_sum_u64(sum);
  __shared__ unsigned long long s_part[kSmallTile / 64];
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < kSmallTile / 64; ++w) t += s_part[w];
    tile_sums[blockIdx.x] = t;
  }
}

// Inclusive prefix of the (at most 4096) tile sums: one block, four consecutive values per thread.
__global__ void __launch_bounds__(kSmallTilesMax / 4)
sample_small_prefix_kernel(const unsigned long long* __restrict__ tile_sums, int n_tiles,
                           unsigned long long* __restrict__ tile_prefix) {
  constexpr int THREADS = kSmallTilesMax / 4, PER = 4;
  pdl_release();
  pdl_wait();
  unsigned long long v[PER], run = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = threadIdx.x * PER + j;
    v[j] = i < n_tiles ? tile_sums[i] : 0ull;
    run += v[j];
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned long long incl = warp_incl_scan_u64(run, lane);
  __shared__ unsigned long long s_warp[THREADS / 32];
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  unsigned long long before = incl - run;
  for (int w = 0; w < warp; ++w) before += s_warp[w];
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = threadIdx.x * PER + j;
    before += v[j];
    if (i < n_tiles) tile_prefix[i] = before;
  }
}

constexpr int kSearchSmallThreads = 256;        // 8 warps, one draw each

// One warp per uniform: a two-level 64-ary search of the inclusive prefix of the tile sums (at most
// 4096 values, L2-resident: two dependent reads), one read of the tile's 256 entries (eight per lane),
// warp scan.  The winner is entered as an integer maximum into first_draw[id] (the earliest draw of a
// prompt has the largest M - k) and the draw remembers where to look (slot_of[k] = id).
__global__ void __launch_bounds__(kSearchSmallThreads, 8)
sample_search_small_kernel(const float* __restrict__ ab, int64_t N, float eps, const float* __restrict__ uniforms,
                           int32_t M, const unsigned long long* __restrict__ pre, int n_tiles,
                           int32_t* __restrict__ cand, int32_t* __restrict__ slot_of, int32_t* first_draw,
                           int32_t* d_status) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = blockIdx.x * (kSearchSmallThreads / 32) + warp;
  pdl_release();
  if (k >= M) return;
  const float u = uniforms[k];                   // an input: read before waiting for the prefix
  pdl_wait();
  // level 1: 64 probes at the ends of 64 equal spans of the prefix (two per lane); they do not depend
  // on the uniform, so they are in flight together with it
  const int span = (n_tiles + 63) >> 6;
  const int i_a = min((2 * lane + 1) * span, n_tiles) - 1, i_b = min((2 * lane + 2) * span, n_tiles) - 1;
  const unsigned long long p_a = pre[i_a], p_b = pre[i_b];
  const unsigned long long wtot = __shfl_sync(0xffffffffu, p_b, 31);           // pre[n_tiles - 1]
  if (wtot == 0 || !(u >= 0.0f) || !(u < 1.0f)) {
    if (lane == 0) {
      cand[k] = -1;
      if (wtot != 0) flag(d_status, SPO_DEV_NONFINITE);
      else if (k == 0) flag(d_status, SPO_DEV_ZERO_TOTAL_WEIGHT);
    }
    return;
  }
  const unsigned long long bigu = __float2ull_rz(u * 4294967296.0f);          // floor(u * 2^32), exact
  const unsigned long long t = (__umul64hi(bigu, wtot) << 32) | ((bigu * wtot) >> 32);
  // first span whose last prefix exceeds t (t < wtot, so there is one); the sum before it
  const unsigned hit_a = __ballot_sync(0xffffffffu, p_a > t), hit_b = __ballot_sync(0xffffffffu, p_b > t);
  const int fa = hit_a ? __ffs(hit_a) - 1 : 32, fb = __ffs(hit_b) - 1;        // spans 2 fa and 2 fb + 1
  const int sp = (fa <= fb) ? 2 * fa : 2 * fb + 1;
  // prefix at the end of span sp - 1: lane (sp-1)/2 holds it (p_a for an even span index, p_b for an odd one)
  unsigned long long before_span = 0ull;
  {
    const unsigned long long from_a = __shfl_sync(0xffffffffu, p_a, sp > 0 ? (sp - 1) >> 1 : 0);
    const unsigned long long from_b = __shfl_sync(0xffffffffu, p_b, sp > 0 ? (sp - 1) >> 1 : 0);
    if (sp > 0) before_span = ((sp - 1) & 1) ? from_b : from_a;
  }
  // level 2: the span's own entries (at most 64: two per lane)
  const int lo = sp * span, n = min(span, n_tiles - lo);
  const unsigned long long q_a = lane < n ? pre[lo + lane] : ~0ull;
  const unsigned long long q_b = lane + 32 < n ? pre[lo + 32 + lane] : ~0ull;
  const unsigned h_a = __ballot_sync(0xffffffffu, q_a > t), h_b = __ballot_sync(0xffffffffu, q_b > t);
  const int off_t = h_a ? __ffs(h_a) - 1 : 32 + __ffs(h_b) - 1;
  const int tile = lo + off_t;
  unsigned long long run = before_span;                                        // sum of all tiles before `tile`
  if (off_t > 0) {
    const unsigned long long r_a = __shfl_sync(0xffffffffu, q_a, (off_t - 1) & 31);
    const unsigned long long r_b = __shfl_sync(0xffffffffu, q_b, (off_t - 1) & 31);
    run = off_t - 1 < 32 ? r_a : r_b;
  }
  // the tile's entries: eight consecutive ones per lane
  const int64_t base = (int64_t)tile * kSmallTile;
  const int n_here = (int)(N - base < kSmallTile ? N - base : kSmallTile);
  const int i0 = 8 * lane;
  unsigned long long q[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) q[j] = 0ull;
  if (i0 + 7 < n_here) {
    const float4* ab4 = reinterpret_cast<const float4*>(ab) + (base + i0) / 2;
    float4 e[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) e[j] = __ldg(ab4 + j);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      q[2 * j] = quantise(entry_weight(e[j].x, e[j].y, eps, d_status));
      q[2 * j + 1] = quantise(entry_weight(e[j].z, e[j].w, eps, d_status));
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (i0 + j < n_here) q[j] = quantise(entry_weight(ab[2 * (base + i0 + j)], ab[2 * (base + i0 + j) + 1], eps, d_status));
  }
  unsigned long long mine = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) mine += q[j];
  const unsigned long long incl = warp_incl_scan_u64(mine, lane);
  const unsigned hit = __ballot_sync(0xffffffffu, run + incl > t);
  int32_t found = -1;
  if (hit) {
    const int first = __ffs(hit) - 1;
    unsigned long long r0 = run + __shfl_sync(0xffffffffu, incl - mine, first);
    int j = 7;
#pragma unroll
    for (int jj = 0; jj < 7; ++jj) {
      r0 += __shfl_sync(0xffffffffu, q[jj], first);
      if (j == 7 && r0 > t) j = jj;
    }
    found = (int32_t)(base + 8 * first + j);
  }
  if (lane == 0) {
    cand[k] = found;
    if (found >= 0) {
      atomicMax(&first_draw[found], M - k);
      slot_of[k] = found;
    }
  }
}

// Keep the first occurrence of every candidate, in order, until B are accepted.  One block;
// each pass covers 8192 draws, eight consecutive ones per thread.  A draw is the first occurrence of
// its prompt when the hash slot the search left it in still holds its own M - k (the largest wins).
__global__ void __launch_bounds__(1024)
sample_accept_kernel(const int32_t* __restrict__ cand, const int32_t* __restrict__ slot_of, int32_t M, int32_t B,
                     const int32_t* __restrict__ vals, int32_t* __restrict__ out_ids, int32_t* d_status) {
  constexpr int PER = 8;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ int s_warp[32];
  __shared__ int s_total;
  if (tid == 0) s_total = 0;
  pdl_wait();                                      // (returns at once when launched the ordinary way)
  __syncthreads();
  for (int k0 = 0; k0 < M; k0 += 1024 * PER) {
    const int base_count = s_total;
    if (base_count >= B) break;
    int32_t c[PER], sl[PER], best[PER];
    const int kt = k0 + tid * PER;
    if (kt + PER <= M) {                           // two 16-byte loads per array
      const int4 c0 = *reinterpret_cast<const int4*>(cand + kt), c1 = *reinterpret_cast<const int4*>(cand + kt + 4);
      const int4 s0 = *reinterpret_cast<const int4*>(slot_of + kt), s1 = *reinterpret_cast<const int4*>(slot_of + kt + 4);
      c[0] = c0.x; c[1] = c0.y; c[2] = c0.z; c[3] = c0.w; c[4] = c1.x; c[5] = c1.y; c[6] = c1.z; c[7] = c1.w;
      sl[0] = s0.x; sl[1] = s0.y; sl[2] = s0.z; sl[3] = s0.w; sl[4] = s1.x; sl[5] = s1.y; sl[6] = s1.z; sl[7] = s1.w;
    } else {
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        c[j] = kt + j < M ? cand[kt + j] : -1;
        sl[j] = kt + j < M ? slot_of[kt + j] : 0;
      }
    }
#pragma unroll
    for (int j = 0; j < PER; ++j) best[j] = c[j] >= 0 ? __ldg(vals + sl[j]) : 0;     // eight independent reads
    bool first[PER];
    int mine = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      first[j] = c[j] >= 0 && best[j] == M - (kt + j);
      mine += first[j];
    }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    int pos = base_count + before + incl - mine;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (first[j]) {
        if (pos < B) out_ids[pos] = c[j];
        ++pos;
      }
    }
    __syncthreads();
    if (tid == 1023) s_total = pos;
    __syncthreads();
  }
  const int accepted = s_total;
  if (accepted < B) {
    for (int i = accepted + tid; i < B; i += 1024) out_ids[i] = -1;
    if (tid == 0) flag(d_status, SPO_DEV_UNIFORMS_EXHAUSTED);
  }
}

// One table entry fetched by id.  Gathers by random id use 8 of the bytes that come back; the
// 64-byte prefetch-size hint keeps L2 from fetching a wider span from HBM for each of them.
__device__ __forceinline__ float2 load_entry(const float2* p) {
  float2 v;
  asm volatile("ld.global.L2::64B.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p));
  return v;
}

// ---------------------------------------------------------------------------
// Advantages: A = r - alpha/(alpha+beta) gathered by id; batch mean / std; normalise.
// ---------------------------------------------------------------------------
// Estimate of one entry, alpha/(alpha+beta); 0.5 for an empty entry.  A negative or non-finite
// entry is reported through `bad_entry` (the caller skips the element).
__device__ __forceinline__ float entry_estimate(float2 e, bool& bad_entry) {
  const float n = e.x + e.y;
  if ((fminf(e.x, e.y) < 0.0f) | !(n < CUDART_INF_F)) { bad_entry = true; return 0.5f; }
  return n > 0.0f ? e.x / n : 0.5f;
}

// Batch statistics carried through the reductions: sum, sum of squares, and the two near-zero
// counts (as doubles: exact, and they ride the same shuffles).
struct AdvSums { double sum, sumsq, n_lo, n_hi; };

__device__ __forceinline__ void adv_accumulate(AdvSums& s, float a, float tau_lo, float tau_hi) {
  s.sum += a;
  s.sumsq += (double)a * a;
  const float m = fabsf(a);
  s.n_lo += m <= tau_lo ? 1.0 : 0.0;
  s.n_hi += m <= tau_hi ? 1.0 : 0.0;
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum of the batch statistics (fixed order); result valid in every thread.
// s_buf: THREADS / 32 entries of shared memory.
template <int THREADS>
__device__ __forceinline__ void block_sum_adv(AdvSums& v, AdvSums* s_buf) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v.sum = warp_sum_f64(v.sum);
  v.sumsq = warp_sum_f64(v.sumsq);
  v.n_lo = warp_sum_f64(v.n_lo);
  v.n_hi = warp_sum_f64(v.n_hi);
  if (lane == 0) s_buf[warp] = v;
  __syncthreads();
  AdvSums t = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) {
    t.sum += s_buf[w].sum; t.sumsq += s_buf[w].sumsq; t.n_lo += s_buf[w].n_lo; t.n_hi += s_buf[w].n_hi;
  }
  v = t;
  __syncthreads();
}

__device__ __forceinline__ void write_stats(float* stats, float mu, float sigma, int32_t B, float m2, const AdvSums& t) {
  stats[0] = mu; stats[1] = sigma; stats[2] = (float)B; stats[3] = m2;
  stats[4] = (float)t.n_lo; stats[5] = (float)t.n_hi; stats[6] = 0.0f; stats[7] = 0.0f;
}


// What the fused advantage + update kernels need besides the advantage inputs.
struct UpdateArgs {
  const float* kl;       // [B] per batch entry, or [N] per prompt (kl_is_table)
  int kl_is_table;
  float rho_min, rho_max, inv_d_half;
};

constexpr unsigned kBadId = 1u, kBadValue = 2u;

// One batch element: A = r - v(id) from the table as it stands (Sec. 3.2: the baseline is the
// estimate before this batch's update) and, with UPDATE, the tracker update of the same entry from
// the value just read (Sec. 3.1), so the entry crosses the memory system once per step.
// Out-of-range ids, negative / non-finite entries and non-finite rewards or divergences are
// reported in `bad`; the element then contributes A = 0 and its entry stays untouched.
// The arithmetic of one element once its entry (and divergence) are in registers.
template <bool UPDATE>
__device__ __forceinline__ float advantage_compute(float2* __restrict__ ab, int32_t id, float2 e, float r, float div,
                                                   const UpdateArgs& u, unsigned& bad) {
  bool bad_entry = false;
  const float v = entry_estimate(e, bad_entry);
  if (bad_entry | !(fabsf(r) < CUDART_INF_F)) { bad |= kBadValue; return 0.0f; }
  if (UPDATE) {
    if (isnan(div)) {
      bad |= kBadValue;                      // entry untouched; the advantage itself is well defined
    } else {
      float rho = exp2f(-div * u.inv_d_half);
      rho = fminf(fmaxf(rho, u.rho_min), u.rho_max);
      e.x = fmaf(rho, e.x, r);
      e.y = fmaf(rho, e.y, 1.0f - r);
      ab[id] = e;
    }
  }
  return r - v;
}

template <bool UPDATE>
__device__ __forceinline__ float advantage_element(float2* __restrict__ ab, int64_t N, int32_t id, float r, int64_t j,
                                                   const UpdateArgs& u, unsigned& bad) {
  if (id < 0 || (int64_t)id >= N) { bad |= kBadId; return 0.0f; }
  const float2 e = load_entry(ab + id);
  float div = 0.0f;
  if (UPDATE) div = u.kl_is_table ? __ldg(u.kl + id) : u.kl[j];
  return advantage_compute<UPDATE>(ab, id, e, r, div, u, bad);
}

__device__ __forceinline__ void flag_bad(int32_t* d_status, unsigned bad) {
  if (bad & kBadId) flag(d_status, SPO_DEV_ID_OUT_OF_RANGE);
  if (bad & kBadValue) flag(d_status, SPO_DEV_NONFINITE);
}

__device__ __forceinline__ void mean_sigma(const AdvSums& t, int32_t B, int32_t ddof, float& mu, float& sigma,
                                           float& m2) {
  double m = B > 0 ? t.sum / B : 0.0;
  double ss = t.sumsq - t.sum * m;             // sum (A - mu)^2
  if (ss < 0.0) ss = 0.0;
  int32_t den = B - ddof;
  double var = den > 0 ? ss / den : 0.0;
  mu = (float)m;
  sigma = (float)sqrt(var);
  m2 = (float)ss;
}

struct NormArgs { float norm_eps; int32_t ddof; float tau_lo, tau_hi; };

// Whole batch in one block: one launch for gather, (update,) statistics and normalisation.
template <bool UPDATE>
__global__ void __launch_bounds__(1024)
advantages_single_kernel(float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                         const float* __restrict__ r, int32_t B, float* __restrict__ a_raw,
                         float* __restrict__ a_norm, float* __restrict__ stats, NormArgs na, UpdateArgs u,
                         int32_t* d_status) {
  constexpr int PER = kAdvSingleBlockMax / 1024;
  __shared__ AdvSums s_buf[32];
  float a[PER];
  AdvSums t = {0.0, 0.0, 0.0, 0.0};
  unsigned bad = 0;
  // The one block is bound by memory latency: first every id, reward and divergence of the thread's
  // elements, then all their table entries, are requested together before any is used.
  int32_t id[PER];
  float rew[PER], div[PER];
  float2 e[PER];
  bool live[PER];
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = j * 1024 + threadIdx.x;
    live[j] = i < B;
    id[j] = live[j] ? ids[i] : 0;
    rew[j] = live[j] ? r[i] : 0.0f;
    div[j] = (UPDATE && live[j] && !u.kl_is_table) ? u.kl[i] : 0.0f;
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    e[j] = make_float2(0.0f, 0.0f);
    if (live[j] && (id[j] < 0 || (int64_t)id[j] >= N)) { bad |= kBadId; live[j] = false; }
    if (live[j]) {
      e[j] = load_entry(ab + id[j]);
      if (UPDATE && u.kl_is_table) div[j] = __ldg(u.kl + id[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = j * 1024 + threadIdx.x;
    a[j] = 0.0f;
    if (i < B) {
      if (live[j]) a[j] = advantage_compute<UPDATE>(ab, id[j], e[j], rew[j], div[j], u, bad);
      adv_accumulate(t, a[j], na.tau_lo, na.tau_hi);
      if (a_raw) a_raw[i] = a[j];
    }
  }
  flag_bad(d_status, bad);
  block_sum_adv<1024>(t, s_buf);
  float mu, sigma, m2;
  mean_sigma(t, B, na.ddof, mu, sigma, m2);
  const float inv = 1.0f / (sigma + na.norm_eps);
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int i = j * 1024 + threadIdx.x;
    if (i < B) a_norm[i] = (a[j] - mu) * inv;
  }
  if (stats && threadIdx.x == 0) write_stats(stats, mu, sigma, B, m2, t);
}

// Large batches, pass 1: raw advantages (stored into `tmp`), the update of the entries when fused,
// and per-block statistics.
template <bool UPDATE>
__global__ void __launch_bounds__(256)
advantages_partial_kernel(float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                          const float* __restrict__ r, int32_t B, float* __restrict__ tmp,
                          AdvSums* __restrict__ partials, NormArgs na, UpdateArgs u, int32_t* d_status) {
  __shared__ AdvSums s_buf[8];
  AdvSums t = {0.0, 0.0, 0.0, 0.0};
  unsigned bad = 0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < B; i += (int64_t)gridDim.x * 256) {
    const float a = advantage_element<UPDATE>(ab, N, ids[i], r[i], i, u, bad);
    tmp[i] = a;
    adv_accumulate(t, a, na.tau_lo, na.tau_hi);
  }
  flag_bad(d_status, bad);
  block_sum_adv<256>(t, s_buf);
  if (threadIdx.x == 0) partials[blockIdx.x] = t;
}

// Pass 2: every block folds the partials in the same fixed order, then normalises its span.
__global__ void __launch_bounds__(256)
advantages_normalise_kernel(const AdvSums* __restrict__ partials, int n_partials, const float* tmp,
                            int32_t B, float* a_norm, float* __restrict__ stats, NormArgs na) {
  __shared__ AdvSums s_buf[8];
  AdvSums t = {0.0, 0.0, 0.0, 0.0};
  for (int i = threadIdx.x; i < n_partials; i += 256) {
    const AdvSums p = partials[i];
    t.sum += p.sum; t.sumsq += p.sumsq; t.n_lo += p.n_lo; t.n_hi += p.n_hi;
  }
  block_sum_adv<256>(t, s_buf);
  float mu, sigma, m2;
  mean_sigma(t, B, na.ddof, mu, sigma, m2);
  const float inv = 1.0f / (sigma + na.norm_eps);
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < B; i += (int64_t)gridDim.x * 256)
    a_norm[i] = (tmp[i] - mu) * inv;
  if (stats && blockIdx.x == 0 && threadIdx.x == 0) write_stats(stats, mu, sigma, B, m2, t);
}

// ---------------------------------------------------------------------------
// Tracker update (Sec. 3.1): rho = clamp(2^(-D/D_half)); alpha <- rho*alpha + r; beta <- rho*beta + 1-r
// ---------------------------------------------------------------------------
// Four batch entries per thread, loads issued before any is used, so that four gathers are in
// flight per thread: the kernel is bound by memory latency, not arithmetic.
__global__ void __launch_bounds__(256)
tracker_update_kernel(float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                      const float* __restrict__ r, const float* __restrict__ kl, int kl_is_table, int32_t B,
                      float rho_min, float rho_max, float inv_d_half, int32_t* d_status) {
  constexpr int U = 4;
  const int64_t stride = (int64_t)gridDim.x * 256;
  for (int64_t j0 = (int64_t)blockIdx.x * 256 + threadIdx.x; j0 < B; j0 += U * stride) {
    int32_t id[U];
    float rew[U], div[U];
    float2 e[U];
    bool live[U];
#pragma unroll
    for (int q = 0; q < U; ++q) {
      const int64_t j = j0 + q * stride;
      live[q] = j < B;
      id[q] = live[q] ? ids[j] : 0;
      rew[q] = live[q] ? r[j] : 0.0f;
      div[q] = (live[q] && !kl_is_table) ? kl[j] : 0.0f;
    }
#pragma unroll
    for (int q = 0; q < U; ++q) {
      if (live[q] && (id[q] < 0 || (int64_t)id[q] >= N)) { flag(d_status, SPO_DEV_ID_OUT_OF_RANGE); live[q] = false; }
      if (live[q]) {
        e[q] = load_entry(ab + id[q]);
        if (kl_is_table) div[q] = __ldg(kl + id[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < U; ++q) {
      if (!live[q]) continue;
      if (isnan(rew[q]) || isinf(rew[q]) || isnan(div[q])) { flag(d_status, SPO_DEV_NONFINITE); continue; }
      float rho = exp2f(-div[q] * inv_d_half);
      rho = fminf(fmaxf(rho, rho_min), rho_max);
      e[q].x = fmaf(rho, e[q].x, rew[q]);
      e[q].y = fmaf(rho, e[q].y, 1.0f - rew[q]);
      ab[id[q]] = e[q];
    }
  }
}

// Tracker update for a batch in which a prompt may appear several times (batch SPO: each prompt is
// rolled out G times against a shared baseline).  The occurrences of one prompt are applied in batch
// order, one per round: in every round each prompt's earliest not-yet-applied occurrence wins an
// integer atomicMin and performs its update, so the result does not depend on thread timing.
// One block; keys/cur is an open-addressing table over the distinct ids (keys preset to 0, id+1 stored).
__global__ void __launch_bounds__(1024)
tracker_update_repeats_kernel(float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                              const float* __restrict__ r, const float* __restrict__ kl, int kl_is_table, int32_t B,
                              int32_t* keys, int32_t* cur, int32_t* slot_of, uint32_t slot_mask,
                              float rho_min, float rho_max, float inv_d_half, int32_t* d_status) {
  const int tid = threadIdx.x;
  __shared__ int s_remaining;
  for (int j = tid; j < B; j += 1024) {
    const int32_t id = ids[j];
    int32_t slot = -1;
    if (id < 0 || (int64_t)id >= N) {
      flag(d_status, SPO_DEV_ID_OUT_OF_RANGE);
    } else {
      const float rew = r[j];
      const float div = kl_is_table ? kl[id] : kl[j];
      if (isnan(rew) || isinf(rew) || isnan(div)) {
        flag(d_status, SPO_DEV_NONFINITE);
      } else {
        uint32_t s = hash_id((uint32_t)id) & slot_mask;
        for (uint32_t probe = 0; probe <= slot_mask; ++probe) {
          const int32_t prev = atomicCAS(&keys[s], 0, id + 1);
          if (prev == 0 || prev == id + 1) { slot = (int32_t)s; break; }
          s = (s + 1) & slot_mask;
        }
      }
    }
    slot_of[j] = slot;
  }
  __syncthreads();
  for (int round = 0; round <= B; ++round) {
    if (tid == 0) s_remaining = 0;
    for (int j = tid; j < B; j += 1024) {
      const int32_t slot = slot_of[j];
      if (slot >= 0) cur[slot] = 0x7fffffff;
    }
    __syncthreads();
    for (int j = tid; j < B; j += 1024) {
      const int32_t slot = slot_of[j];
      if (slot >= 0) atomicMin(&cur[slot], j);
    }
    __syncthreads();
    for (int j = tid; j < B; j += 1024) {
      const int32_t slot = slot_of[j];
      if (slot < 0) continue;
      if (__ldcg(&cur[slot]) == j) {                  // read at L2, where the atomics were performed
        const int32_t id = ids[j];
        const float rew = r[j];
        const float div = kl_is_table ? kl[id] : kl[j];
        float rho = exp2f(-div * inv_d_half);
        rho = fminf(fmaxf(rho, rho_min), rho_max);
        float2 e = ab[id];
        e.x = fmaf(rho, e.x, rew);
        e.y = fmaf(rho, e.y, 1.0f - rew);
        ab[id] = e;
        slot_of[j] = -1;
      } else {
        s_remaining = 1;
      }
    }
    __syncthreads();
    if (s_remaining == 0) break;
    __syncthreads();
  }
}

// Normalisation with statistics supplied by the caller (e.g. merged over data-parallel ranks).
__global__ void __launch_bounds__(256)
advantages_apply_kernel(const float* a_raw, int32_t B, float mu, float inv, float* a_norm) {
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < B; i += (int64_t)gridDim.x * 256)
    a_norm[i] = (a_raw[i] - mu) * inv;
}

}  // namespace

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------

SampleWs sample_ws_layout(int64_t N, int32_t M) {
  SampleWs L{};
  L.small = N <= kSmallTableMax ? 1 : 0;
  L.n_tiles = ceil_div(N, L.small ? kSmallTile : kSampleTile);
  L.n_super = L.small ? 1 : (int)ceil_div(L.n_tiles, kSuperTile);
  int64_t slots = 64;
  while (!L.small && slots < 2 * (int64_t)M) slots <<= 1;      // the small form keeps first draws per prompt, no hash table
  L.hash_slots = slots;
  size_t off = 0;
  // one zero-filled region: super-tile sums (small form: the ticket), hash keys, hash values
  L.super_sums = off;   off = align_up(off + sizeof(unsigned long long) * (size_t)L.n_super, 256);
  L.keys = off;         off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
  L.vals = off;         off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
  L.zeroed_bytes = off;
  L.tile_sums = off;    off = align_up(off + sizeof(unsigned long long) * (size_t)L.n_tiles * (L.small ? 2 : 1), 256);
  L.cand = off;         off = align_up(off + sizeof(int32_t) * (size_t)M, 256);
  L.slot_of = off;      off = align_up(off + sizeof(int32_t) * (size_t)M, 256);
  L.first_draw = off;   off = align_up(off + (L.small ? sizeof(int32_t) * (size_t)(N + 1) : 0), 256);
  L.total = off;
  return L;
}

cudaError_t launch_tracker_init(float* ab, const float* v0, int64_t N, float n0, cudaStream_t st) {
  if (N == 0) return cudaSuccess;
  int blocks = (int)(ceil_div(N, 256) < (int64_t)sm_count() * 16 ? ceil_div(N, 256) : (int64_t)sm_count() * 16);
  tracker_init_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float2*>(ab), v0, N, n0);
  return cudaGetLastError();
}

cudaError_t launch_sample(const float* ab, int64_t N, const float* u, int32_t M, int32_t B,
                          int32_t* out_ids, float* out_w, char* ws, const SampleWs& L,
                          float eps, int32_t* d_status, cudaStream_t st) {
  auto* tile_sums = reinterpret_cast<unsigned long long*>(ws + L.tile_sums);
  auto* super_sums = reinterpret_cast<unsigned long long*>(ws + L.super_sums);
  auto* cand = reinterpret_cast<int32_t*>(ws + L.cand);
  auto* slot_of = reinterpret_cast<int32_t*>(ws + L.slot_of);
  auto* keys = reinterpret_cast<int32_t*>(ws + L.keys);
  auto* vals = reinterpret_cast<int32_t*>(ws + L.vals);
  cudaError_t e;
  if (L.small) {
    // four launches, nothing to clear beforehand (the first kernel clears the first-draw array);
    // the prefix of the tile sums sits behind the tile sums themselves
    const float4* ab4 = reinterpret_cast<const float4*>(ab);
    unsigned long long* tile_prefix = tile_sums + L.n_tiles;
    int32_t* first_draw = reinterpret_cast<int32_t*>(ws + L.first_draw);
    if (out_w)
      sample_small_sums_kernel<true><<<(unsigned)L.n_tiles, kSmallTile / 2, 0, st>>>(
          ab4, N, eps, reinterpret_cast<float2*>(out_w), out_w, tile_sums, first_draw, d_status);
    else
      sample_small_sums_kernel<false><<<(unsigned)L.n_tiles, kSmallTile / 2, 0, st>>>(
          ab4, N, eps, nullptr, nullptr, tile_sums, first_draw, d_status);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // the other three may be set up while their predecessor runs (they wait for it on the device)
    cudaLaunchAttribute early[1];
    early[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    early[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = early;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(kSmallTilesMax / 4);
    e = cudaLaunchKernelEx(&cfg, sample_small_prefix_kernel, (const unsigned long long*)tile_sums, (int)L.n_tiles,
                           tile_prefix);
    if (e != cudaSuccess) return e;
    cfg.gridDim = dim3((unsigned)ceil_div(M, kSearchSmallThreads / 32));
    cfg.blockDim = dim3(kSearchSmallThreads);
    e = cudaLaunchKernelEx(&cfg, sample_search_small_kernel, ab, N, eps, u, M, (const unsigned long long*)tile_prefix,
                           (int)L.n_tiles, cand, slot_of, first_draw, d_status);
    if (e != cudaSuccess) return e;
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(1024);
    return cudaLaunchKernelEx(&cfg, sample_accept_kernel, (const int32_t*)cand, (const int32_t*)slot_of, M, B,
                              (const int32_t*)first_draw, out_ids, d_status);
  }
  if ((e = cudaMemsetAsync(ws, 0, L.zeroed_bytes, st)) != cudaSuccess) return e;
  if (out_w)
    sample_tile_sums_kernel<true><<<(unsigned)L.n_tiles, 256, 0, st>>>(
        reinterpret_cast<const float4*>(ab), N, eps, reinterpret_cast<float2*>(out_w), out_w, tile_sums, super_sums,
        d_status);
  else
    sample_tile_sums_kernel<false><<<(unsigned)L.n_tiles, 256, 0, st>>>(
        reinterpret_cast<const float4*>(ab), N, eps, nullptr, nullptr, tile_sums, super_sums, d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  sample_search_kernel<<<(unsigned)ceil_div((int64_t)M * 32, 256), 256, 0, st>>>(
      ab, N, eps, u, M, tile_sums, super_sums, L.n_tiles, L.n_super, cand, slot_of, keys, vals,
      (uint32_t)(L.hash_slots - 1), d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  sample_accept_kernel<<<1, 1024, 0, st>>>(cand, slot_of, M, B, vals, out_ids, d_status);
  return cudaGetLastError();
}

RepeatsWs repeats_ws_layout(int32_t B) {
  RepeatsWs L{};
  int64_t slots = 64;
  while (slots < 2 * (int64_t)B) slots <<= 1;
  L.hash_slots = slots;
  size_t off = 0;
  L.keys = off;    off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
  L.zeroed_bytes = off;
  L.cur = off;     off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
  L.slot_of = off; off = align_up(off + sizeof(int32_t) * (size_t)(B > 0 ? B : 1), 256);
  L.total = off;
  return L;
}

cudaError_t launch_tracker_update_repeats(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                                          int kl_is_table, int32_t B, char* ws, const RepeatsWs& L, float rho_min,
                                          float rho_max, float d_half, int32_t* d_status, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(ws + L.keys, 0, L.zeroed_bytes, st);
  if (e != cudaSuccess) return e;
  tracker_update_repeats_kernel<<<1, 1024, 0, st>>>(
      reinterpret_cast<float2*>(ab), N, ids, r, kl, kl_is_table, B, reinterpret_cast<int32_t*>(ws + L.keys),
      reinterpret_cast<int32_t*>(ws + L.cur), reinterpret_cast<int32_t*>(ws + L.slot_of),
      (uint32_t)(L.hash_slots - 1), rho_min, rho_max, 1.0f / d_half, d_status);
  return cudaGetLastError();
}

cudaError_t launch_advantages_apply(const float* a_raw, int32_t B, float mu, float sigma, float norm_eps, float* a_norm,
                                    cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  advantages_apply_kernel<<<adv_blocks(B), 256, 0, st>>>(a_raw, B, mu, 1.0f / (sigma + norm_eps), a_norm);
  return cudaGetLastError();
}

int adv_blocks(int32_t B) {
  int64_t want = ceil_div(B, 2048);
  int64_t cap = (int64_t)sm_count() * 4;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return (int)want;
}

// Advantages of a batch (and, with `upd`, the tracker update of the same entries in the same pass).
// partials: scratch for adv_blocks(B) block records when B exceeds one block's capacity.
cudaError_t launch_advantages(float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                              float* a_raw, float* a_norm, float* stats, void* partials, const spo_params& pr,
                              const AdvUpdate* upd, bool force_two_pass, int32_t* d_status, cudaStream_t st) {
  float2* ab2 = reinterpret_cast<float2*>(ab);
  const NormArgs na = {pr.norm_eps, pr.norm_ddof, pr.near_zero_tau_lo, pr.near_zero_tau_hi};
  UpdateArgs u = {nullptr, 0, pr.rho_min, pr.rho_max, 1.0f / pr.d_half};
  if (upd) { u.kl = upd->kl; u.kl_is_table = upd->kl_is_table; }
  if (B <= kAdvSingleBlockMax && !force_two_pass) {
    if (upd) advantages_single_kernel<true><<<1, 1024, 0, st>>>(ab2, N, ids, r, B, a_raw, a_norm, stats, na, u, d_status);
    else advantages_single_kernel<false><<<1, 1024, 0, st>>>(ab2, N, ids, r, B, a_raw, a_norm, stats, na, u, d_status);
    return cudaGetLastError();
  }
  const int blocks = adv_blocks(B);
  AdvSums* part = reinterpret_cast<AdvSums*>(partials);
  float* tmp = a_raw ? a_raw : a_norm;
  if (upd) advantages_partial_kernel<true><<<blocks, 256, 0, st>>>(ab2, N, ids, r, B, tmp, part, na, u, d_status);
  else advantages_partial_kernel<false><<<blocks, 256, 0, st>>>(ab2, N, ids, r, B, tmp, part, na, u, d_status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  advantages_normalise_kernel<<<blocks, 256, 0, st>>>(part, blocks, tmp, B, a_norm, stats, na);
  return cudaGetLastError();
}

size_t adv_partial_bytes(int32_t B) { return align_up(sizeof(AdvSums) * (size_t)adv_blocks(B), 256); }

cudaError_t launch_tracker_update(float* ab, int64_t N, const int32_t* ids, const float* r,
                                  const float* kl, int kl_is_table, int32_t B,
                                  float rho_min, float rho_max, float d_half,
                                  int32_t* d_status, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  int64_t blocks = ceil_div(B, 256 * 4);
  int64_t cap = (int64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  tracker_update_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<float2*>(ab), N, ids, r, kl, kl_is_table, B,
                                                          rho_min, rho_max, 1.0f / d_half, d_status);
  return cudaGetLastError();
}

}  // namespace spo

// ---------------------------------------------------------------------------
// spo_advantages_static: the two-pass advantage kernels with their scratch in a
// fixed device array instead of a caller buffer (see include/spo.h).
// ---------------------------------------------------------------------------
namespace spo {
namespace {

constexpr int kStaticAdvMaxBlocks = 1024;

// Per-block statistics records of pass 1.  Lives in every GPU context that loads this
// library, 32 KB, until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) AdvSums g_adv_static_scratch[kStaticAdvMaxBlocks];

std::mutex g_adv_static_mutex;
AdvSums* g_adv_static_ptr[64] = {};

// Device address of the scratch array for the current device (looked up once per device).
cudaError_t adv_static_scratch(AdvSums** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_adv_static_mutex);
  if (!g_adv_static_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_adv_static_scratch);
    if (e != cudaSuccess) return e;
    g_adv_static_ptr[dev] = static_cast<AdvSums*>(ptr);
  }
  *out = g_adv_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace spo

extern "C" int32_t spo_advantages_static(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                                         float* a_raw, float* a_norm, float* stats, const spo_params* params,
                                         int32_t* d_status, void* stream) {
  using namespace spo;
  if (!params || !ab || !ids || !r || !a_norm) return SPO_ERR_INVALID_ARG;
  if (!(params->norm_eps >= 0.0f) || (params->norm_ddof != 0 && params->norm_ddof != 1)) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31) || B < 1) return SPO_ERR_BAD_SHAPE;
  if (B > SPO_ADVANTAGES_STATIC_MAX_B) return SPO_ERR_BAD_SHAPE;   // beyond what the fixed scratch is sized for
  const uintptr_t all = reinterpret_cast<uintptr_t>(ab) | reinterpret_cast<uintptr_t>(ids) |
                        reinterpret_cast<uintptr_t>(r) | reinterpret_cast<uintptr_t>(a_raw) |
                        reinterpret_cast<uintptr_t>(a_norm) | reinterpret_cast<uintptr_t>(stats);
  if (all & 15u) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  AdvSums* partials = nullptr;
  cudaError_t e = adv_static_scratch(&partials);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (adv_blocks(B) > kStaticAdvMaxBlocks) return SPO_ERR_BAD_SHAPE;
  // Pass 1 overwrites partials[0..blocks) and pass 2 reads exactly those, so nothing left
  // over from an earlier call is ever read and nothing needs clearing.
  e = launch_advantages(const_cast<float*>(ab), N, ids, r, B, a_raw, a_norm, stats, partials, *params, nullptr,
                        /*force_two_pass=*/true, d_status, (cudaStream_t)stream);
  if (e != cudaSuccess) return record_cuda_error(e);
  return SPO_OK;
}
