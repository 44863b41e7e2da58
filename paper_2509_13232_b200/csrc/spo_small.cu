// Tracker, advantage and sampling kernels: the small group-free pieces of SPO.
// All are memory-streaming kernels: coalesced vector loads of the interleaved
// (alpha, beta) table, warp-shuffle reductions, integer prefix sums.
#include <cuda_runtime.h>
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
// Sampling weight of one table entry (Eq. "sampling_coef") in IEEE fp32, one
// rounded operation per step so that a host restatement gives the same bits:
// n=a+b, num=a*b, den=n*n, p=num/den (0.25 for an empty entry), s=sqrt(p), w=s+eps.
// A negative or non-finite entry yields weight 0 and *bad = true.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float entry_weight(float a, float b, float eps, bool& bad) {
  if (!(a >= 0.0f) || !(b >= 0.0f) || isinf(a) || isinf(b)) { bad = true; return 0.0f; }
  float n = __fadd_rn(a, b);
  float p = 0.25f;
  if (n > 0.0f) p = __fdiv_rn(__fmul_rn(a, b), __fmul_rn(n, n));
  return __fadd_rn(__fsqrt_rn(p), eps);
}

// q = floor(w * 2^32): exact, the scale is a power of two.
__device__ __forceinline__ unsigned long long quantise(float w) {
  return (unsigned long long)((double)w * 4294967296.0);
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
__global__ void __launch_bounds__(256)
sample_tile_sums_kernel(const float4* __restrict__ ab4, int64_t N, float eps, float2* __restrict__ out_w2,
                        float* __restrict__ out_w, unsigned long long* __restrict__ tile_sums,
                        int32_t* d_status) {
  const int64_t tile = blockIdx.x;
  const int64_t first_pair = tile * (kSampleTile / 2);
  const int64_t n_pairs = N >> 1;
  unsigned long long sum = 0;
  bool bad = false;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int64_t p = first_pair + j * 256 + threadIdx.x;
    if (p < n_pairs) {
      float4 e = __ldg(ab4 + p);
      float w0 = entry_weight(e.x, e.y, eps, bad);
      float w1 = entry_weight(e.z, e.w, eps, bad);
      sum += quantise(w0) + quantise(w1);
      if (out_w2) out_w2[p] = make_float2(w0, w1);
    } else if (p == n_pairs && (N & 1)) {      // odd tail entry
      const float* ab = reinterpret_cast<const float*>(ab4);
      float w0 = entry_weight(ab[2 * (N - 1)], ab[2 * (N - 1) + 1], eps, bad);
      sum += quantise(w0);
      if (out_w) out_w[N - 1] = w0;
    }
  }
  sum = warp_sum_u64(sum);
  __shared__ unsigned long long s_part[8];
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = sum;
  if (__syncthreads_or(bad) && threadIdx.x == 0) flag(d_status, SPO_DEV_NONFINITE);
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += s_part[w];
    tile_sums[tile] = t;
  }
}

// Exclusive scan of the tile sums by one block; offsets[n_tiles] = total weight.
__global__ void __launch_bounds__(1024)
sample_scan_tiles_kernel(const unsigned long long* __restrict__ tile_sums, int64_t n_tiles,
                         unsigned long long* __restrict__ offsets, int32_t* d_status) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t per = (n_tiles + 1023) / 1024;
  const int64_t lo = (int64_t)tid * per;
  const int64_t hi = lo + per < n_tiles ? lo + per : n_tiles;
  unsigned long long local = 0;
  for (int64_t i = lo; i < hi; ++i) local += tile_sums[i];
  unsigned long long incl = warp_incl_scan_u64(local, lane);
  __shared__ unsigned long long s_warp[32];
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    unsigned long long v = s_warp[lane];
    unsigned long long s = warp_incl_scan_u64(v, lane);
    s_warp[lane] = s - v;                       // exclusive prefix of the warp totals
    if (lane == 31) {
      offsets[n_tiles] = s;
      if (s == 0) flag(d_status, SPO_DEV_ZERO_TOTAL_WEIGHT);
    }
  }
  __syncthreads();
  unsigned long long run = s_warp[warp] + incl - local;
  for (int64_t i = lo; i < hi; ++i) {
    offsets[i] = run;
    run += tile_sums[i];
  }
}

// One warp per uniform: threshold, tile by binary search, entry by a scan inside the tile.
__global__ void __launch_bounds__(256)
sample_search_kernel(const float* __restrict__ ab, int64_t N, float eps, const float* __restrict__ uniforms,
                     int32_t M, const unsigned long long* __restrict__ offsets, int64_t n_tiles,
                     int32_t* __restrict__ cand, int32_t* d_status) {
  const int lane = threadIdx.x & 31;
  const int k = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (k >= M) return;
  const unsigned long long wtot = offsets[n_tiles];
  const float u = uniforms[k];
  if (wtot == 0 || !(u >= 0.0f) || !(u < 1.0f)) {
    if (lane == 0) {
      cand[k] = -1;
      if (wtot != 0) flag(d_status, SPO_DEV_NONFINITE);
    }
    return;
  }
  const unsigned long long bigu = (unsigned long long)((double)u * 4294967296.0);
  const unsigned long long t = (__umul64hi(bigu, wtot) << 32) | ((bigu * wtot) >> 32);
  // first tile j with offsets[j+1] > t
  int64_t lo = 0, hi = n_tiles - 1;
  while (lo < hi) {
    int64_t mid = (lo + hi) >> 1;
    if (offsets[mid + 1] > t) hi = mid; else lo = mid + 1;
  }
  unsigned long long run = offsets[lo];
  const int64_t base = lo * kSampleTile;
  int32_t found = -1;
  bool bad = false;
  for (int c = 0; c < kSampleTile / 32; ++c) {
    int64_t i = base + c * 32 + lane;
    unsigned long long q = 0;
    if (i < N) q = quantise(entry_weight(ab[2 * i], ab[2 * i + 1], eps, bad));
    unsigned long long incl = warp_incl_scan_u64(q, lane);
    unsigned hit = __ballot_sync(0xffffffffu, run + incl > t);
    if (hit) { found = (int32_t)(base + c * 32 + (__ffs(hit) - 1)); break; }
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) cand[k] = found;
}

__device__ __forceinline__ uint32_t hash_id(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

// Keep the first occurrence of every candidate, in order, until B are accepted.
// One block; keys/vals is an open-addressing table (keys preset to -1, vals to 0x7f7f7f7f).
__global__ void __launch_bounds__(1024)
sample_accept_kernel(const int32_t* __restrict__ cand, int32_t M, int32_t B, int32_t* __restrict__ keys,
                     int32_t* __restrict__ vals, uint32_t slot_mask, int32_t* __restrict__ out_ids,
                     int32_t* d_status) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int k = tid; k < M; k += 1024) {
    int32_t c = cand[k];
    if (c < 0) continue;
    uint32_t s = hash_id((uint32_t)c) & slot_mask;
    for (uint32_t probe = 0; probe <= slot_mask; ++probe) {
      int32_t prev = atomicCAS(&keys[s], -1, c);
      if (prev == -1 || prev == c) { atomicMin(&vals[s], k); break; }
      s = (s + 1) & slot_mask;
    }
  }
  __syncthreads();
  __shared__ int s_warp[32];
  __shared__ int s_total;
  if (tid == 0) s_total = 0;
  __syncthreads();
  for (int k0 = 0; k0 < M; k0 += 1024) {
    const int base_count = s_total;
    if (base_count >= B) break;
    const int k = k0 + tid;
    int first = 0;
    int32_t c = -1;
    if (k < M) {
      c = cand[k];
      if (c >= 0) {
        uint32_t s = hash_id((uint32_t)c) & slot_mask;
        for (uint32_t probe = 0; probe <= slot_mask; ++probe) {
          if (keys[s] == c) { first = (vals[s] == k); break; }
          s = (s + 1) & slot_mask;
        }
      }
    }
    unsigned bal = __ballot_sync(0xffffffffu, first);
    int in_warp = __popc(bal & ((1u << lane) - 1));
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    int pos = base_count + before + in_warp;
    if (first && pos < B) out_ids[pos] = c;
    __syncthreads();
    if (tid == 1023) s_total = pos + first;
    __syncthreads();
  }
  const int accepted = s_total;
  if (accepted < B) {
    for (int i = accepted + tid; i < B; i += 1024) out_ids[i] = -1;
    if (tid == 0) flag(d_status, SPO_DEV_UNIFORMS_EXHAUSTED);
  }
}

// ---------------------------------------------------------------------------
// Advantages: A = r - alpha/(alpha+beta) gathered by id; batch mean / std; normalise.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float gather_advantage(const float2* __restrict__ ab, int64_t N, int32_t id, float r,
                                                  bool& bad_id) {
  if (id < 0 || (int64_t)id >= N) { bad_id = true; return 0.0f; }
  float2 e = __ldg(ab + id);
  float n = e.x + e.y;
  float v = n > 0.0f ? e.x / n : 0.5f;
  return r - v;
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum of two doubles; result valid in every thread.
template <int THREADS>
__device__ __forceinline__ void block_sum2(double& a, double& b, double* s_a, double* s_b) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  a = warp_sum_f64(a);
  b = warp_sum_f64(b);
  if (lane == 0) { s_a[warp] = a; s_b[warp] = b; }
  __syncthreads();
  double ta = 0.0, tb = 0.0;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) { ta += s_a[w]; tb += s_b[w]; }
  a = ta; b = tb;
  __syncthreads();
}

__device__ __forceinline__ void mean_sigma(double sum, double sumsq, int32_t B, int32_t ddof, float& mu, float& sigma) {
  double m = B > 0 ? sum / B : 0.0;
  double ss = sumsq - sum * m;                 // sum (A - mu)^2
  if (ss < 0.0) ss = 0.0;
  int32_t den = B - ddof;
  double var = den > 0 ? ss / den : 0.0;
  mu = (float)m;
  sigma = (float)sqrt(var);
}

// Whole batch in one block: one launch for gather, statistics and normalisation.
__global__ void __launch_bounds__(1024)
advantages_single_kernel(const float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                         const float* __restrict__ r, int32_t B, float* __restrict__ a_raw,
                         float* __restrict__ a_norm, float* __restrict__ stats, float norm_eps, int32_t ddof,
                         int32_t* d_status) {
  constexpr int PER = kAdvSingleBlockMax / 1024;
  __shared__ double s_a[32], s_b[32];
  float a[PER];
  double sum = 0.0, sumsq = 0.0;
  bool bad = false;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int i = j * 1024 + threadIdx.x;
    a[j] = 0.0f;
    if (i < B) {
      a[j] = gather_advantage(ab, N, ids[i], r[i], bad);
      sum += a[j];
      sumsq += (double)a[j] * a[j];
      if (a_raw) a_raw[i] = a[j];
    }
  }
  if (bad) flag(d_status, SPO_DEV_ID_OUT_OF_RANGE);
  block_sum2<1024>(sum, sumsq, s_a, s_b);
  float mu, sigma;
  mean_sigma(sum, sumsq, B, ddof, mu, sigma);
  const float inv = 1.0f / (sigma + norm_eps);
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int i = j * 1024 + threadIdx.x;
    if (i < B) a_norm[i] = (a[j] - mu) * inv;
  }
  if (stats && threadIdx.x == 0) { stats[0] = mu; stats[1] = sigma; stats[2] = (float)B; stats[3] = 0.0f; }
}

// Large batches, pass 1: raw advantages (stored into `tmp`) and per-block (sum, sum of squares).
__global__ void __launch_bounds__(256)
advantages_partial_kernel(const float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                          const float* __restrict__ r, int32_t B, float* __restrict__ tmp,
                          double2* __restrict__ partials, int32_t* d_status) {
  __shared__ double s_a[8], s_b[8];
  double sum = 0.0, sumsq = 0.0;
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < B; i += (int64_t)gridDim.x * 256) {
    float a = gather_advantage(ab, N, ids[i], r[i], bad);
    tmp[i] = a;
    sum += a;
    sumsq += (double)a * a;
  }
  if (bad) flag(d_status, SPO_DEV_ID_OUT_OF_RANGE);
  block_sum2<256>(sum, sumsq, s_a, s_b);
  if (threadIdx.x == 0) partials[blockIdx.x] = make_double2(sum, sumsq);
}

// Pass 2: every block folds the partials in the same fixed order, then normalises its span.
__global__ void __launch_bounds__(256)
advantages_normalise_kernel(const double2* __restrict__ partials, int n_partials, const float* tmp,
                            int32_t B, float* a_norm, float* __restrict__ stats, float norm_eps,
                            int32_t ddof) {
  __shared__ double s_a[8], s_b[8];
  double sum = 0.0, sumsq = 0.0;
  for (int i = threadIdx.x; i < n_partials; i += 256) {
    double2 p = partials[i];
    sum += p.x;
    sumsq += p.y;
  }
  block_sum2<256>(sum, sumsq, s_a, s_b);
  float mu, sigma;
  mean_sigma(sum, sumsq, B, ddof, mu, sigma);
  const float inv = 1.0f / (sigma + norm_eps);
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < B; i += (int64_t)gridDim.x * 256)
    a_norm[i] = (tmp[i] - mu) * inv;
  if (stats && blockIdx.x == 0 && threadIdx.x == 0) {
    stats[0] = mu; stats[1] = sigma; stats[2] = (float)B; stats[3] = 0.0f;
  }
}

// ---------------------------------------------------------------------------
// Tracker update (Sec. 3.1): rho = clamp(2^(-D/D_half)); alpha <- rho*alpha + r; beta <- rho*beta + 1-r
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
tracker_update_kernel(float2* __restrict__ ab, int64_t N, const int32_t* __restrict__ ids,
                      const float* __restrict__ r, const float* __restrict__ kl, int kl_is_table, int32_t B,
                      float rho_min, float rho_max, float inv_d_half, int32_t* d_status) {
  for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < B; j += (int64_t)gridDim.x * 256) {
    const int32_t id = ids[j];
    if (id < 0 || (int64_t)id >= N) { flag(d_status, SPO_DEV_ID_OUT_OF_RANGE); continue; }
    const float rew = r[j];
    const float div = kl_is_table ? __ldg(kl + id) : kl[j];
    if (isnan(rew) || isinf(rew) || isnan(div)) { flag(d_status, SPO_DEV_NONFINITE); continue; }
    float rho = exp2f(-div * inv_d_half);
    rho = fminf(fmaxf(rho, rho_min), rho_max);
    float2 e = ab[id];
    e.x = fmaf(rho, e.x, rew);
    e.y = fmaf(rho, e.y, 1.0f - rew);
    ab[id] = e;
  }
}

}  // namespace

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------

SampleWs sample_ws_layout(int64_t N, int32_t M) {
  SampleWs L{};
  L.n_tiles = ceil_div(N, kSampleTile);
  int64_t slots = 64;
  while (slots < 2 * (int64_t)M) slots <<= 1;
  L.hash_slots = slots;
  size_t off = 0;
  L.tile_sums = off;    off = align_up(off + sizeof(unsigned long long) * L.n_tiles, 256);
  L.tile_offsets = off; off = align_up(off + sizeof(unsigned long long) * (L.n_tiles + 1), 256);
  L.cand = off;         off = align_up(off + sizeof(int32_t) * (size_t)M, 256);
  L.keys = off;         off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
  L.vals = off;         off = align_up(off + sizeof(int32_t) * (size_t)slots, 256);
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
  auto* offsets = reinterpret_cast<unsigned long long*>(ws + L.tile_offsets);
  auto* cand = reinterpret_cast<int32_t*>(ws + L.cand);
  auto* keys = reinterpret_cast<int32_t*>(ws + L.keys);
  auto* vals = reinterpret_cast<int32_t*>(ws + L.vals);
  cudaError_t e;
  if ((e = cudaMemsetAsync(keys, 0xFF, sizeof(int32_t) * L.hash_slots, st)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(vals, 0x7F, sizeof(int32_t) * L.hash_slots, st)) != cudaSuccess) return e;
  sample_tile_sums_kernel<<<(unsigned)L.n_tiles, 256, 0, st>>>(
      reinterpret_cast<const float4*>(ab), N, eps, reinterpret_cast<float2*>(out_w), out_w, tile_sums, d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  sample_scan_tiles_kernel<<<1, 1024, 0, st>>>(tile_sums, L.n_tiles, offsets, d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  sample_search_kernel<<<(unsigned)ceil_div((int64_t)M * 32, 256), 256, 0, st>>>(
      ab, N, eps, u, M, offsets, L.n_tiles, cand, d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  sample_accept_kernel<<<1, 1024, 0, st>>>(cand, M, B, keys, vals, (uint32_t)(L.hash_slots - 1), out_ids, d_status);
  return cudaGetLastError();
}

int adv_blocks(int32_t B) {
  int64_t want = ceil_div(B, 2048);
  int64_t cap = (int64_t)sm_count() * 4;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return (int)want;
}

cudaError_t launch_advantages(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                              float* a_raw, float* a_norm, float* stats, char* ws,
                              float norm_eps, int32_t ddof, int32_t* d_status, cudaStream_t st) {
  const float2* ab2 = reinterpret_cast<const float2*>(ab);
  if (B <= kAdvSingleBlockMax) {
    advantages_single_kernel<<<1, 1024, 0, st>>>(ab2, N, ids, r, B, a_raw, a_norm, stats, norm_eps, ddof, d_status);
    return cudaGetLastError();
  }
  const int blocks = adv_blocks(B);
  double2* partials = reinterpret_cast<double2*>(ws);
  float* tmp = a_raw ? a_raw : a_norm;
  advantages_partial_kernel<<<blocks, 256, 0, st>>>(ab2, N, ids, r, B, tmp, partials, d_status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  advantages_normalise_kernel<<<blocks, 256, 0, st>>>(partials, blocks, tmp, B, a_norm, stats, norm_eps, ddof);
  return cudaGetLastError();
}

cudaError_t launch_tracker_update(float* ab, int64_t N, const int32_t* ids, const float* r,
                                  const float* kl, int kl_is_table, int32_t B,
                                  float rho_min, float rho_max, float d_half,
                                  int32_t* d_status, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  int64_t blocks = ceil_div(B, 256);
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

// Per-block (sum, sum of squares) partials of pass 1.  Lives in every GPU context that
// loads this library, 16 KB, until the process exits.  In host code this name is only a
// handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) double2 g_adv_static_scratch[kStaticAdvMaxBlocks];

std::mutex g_adv_static_mutex;
double2* g_adv_static_ptr[64] = {};

// Device address of the scratch array for the current device (looked up once per device).
cudaError_t adv_static_scratch(double2** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_adv_static_mutex);
  if (!g_adv_static_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_adv_static_scratch);
    if (e != cudaSuccess) return e;
    g_adv_static_ptr[dev] = static_cast<double2*>(ptr);
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
  double2* partials = nullptr;
  cudaError_t e = adv_static_scratch(&partials);
  if (e != cudaSuccess) return SPO_ERR_CUDA;
  int blocks = adv_blocks(B);
  if (blocks > kStaticAdvMaxBlocks) blocks = kStaticAdvMaxBlocks;
  cudaStream_t st = (cudaStream_t)stream;
  const float2* ab2 = reinterpret_cast<const float2*>(ab);
  float* tmp = a_raw ? a_raw : a_norm;
  // Pass 1 overwrites partials[0..blocks) and pass 2 reads exactly those, so nothing left
  // over from an earlier call is ever read and nothing needs clearing.
  advantages_partial_kernel<<<blocks, 256, 0, st>>>(ab2, N, ids, r, B, tmp, partials, d_status);
  if ((e = cudaGetLastError()) != cudaSuccess) return SPO_ERR_CUDA;
  advantages_normalise_kernel<<<blocks, 256, 0, st>>>(partials, blocks, tmp, B, a_norm, stats, params->norm_eps,
                                                      params->norm_ddof);
  if ((e = cudaGetLastError()) != cudaSuccess) return SPO_ERR_CUDA;
  return SPO_OK;
}
