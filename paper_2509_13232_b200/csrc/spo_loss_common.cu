// Loss pieces shared by both element types (token count, per-token finalisation of the
// clipped surrogate, per-response sums) and the plain fp32 SIMT forward / backward used
// for fp32 inputs.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "spo_internal.h"

namespace spo {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void flag(int32_t* d_status, int bit) {
  if (d_status) atomicOr(d_status, bit);
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// counters[0] = number of unmasked token rows
__global__ void __launch_bounds__(256)
count_mask_kernel(const uint8_t* __restrict__ mask, int64_t T, int32_t* counters) {
  int local = 0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < T; i += (int64_t)gridDim.x * 256)
    local += mask[i] != 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(&counters[0], local);
}

__global__ void set_count_kernel(int32_t value, int32_t* counters) { counters[0] = value; }

// Sequence-mean aggregation: seq_cnt[s] = unmasked tokens of response s; counters[2] = responses
// that have at least one.
__global__ void __launch_bounds__(256)
seq_count_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu_seqlens, int32_t* __restrict__ seq_cnt,
                 int32_t* counters) {
  const int s = blockIdx.x;
  const int64_t lo = cu_seqlens[s], hi = cu_seqlens[s + 1];
  int local = 0;
  if (mask) {
    for (int64_t t = lo + threadIdx.x; t < hi; t += 256) local += mask[t] != 0;
  } else if (threadIdx.x == 0) {
    local = (int)(hi - lo);
  }
  __shared__ int s_w[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_w[w];
    seq_cnt[s] = tot;
    if (tot > 0) atomicAdd(&counters[2], 1);
  }
}

// Per token: merge the vocabulary splits' (max, sum-exp, target logit), then the
// importance ratio, the clipped surrogate (Sec. 3.2) and d loss / d logp.
__global__ void __launch_bounds__(kFinalizeThreads)
fwd_finalize_kernel(const FwdPartial* __restrict__ partials, int nsplit, const int32_t* __restrict__ y,
                    const float* __restrict__ logp_old, const uint8_t* __restrict__ mask,
                    const int32_t* __restrict__ cu_seqlens, const float* __restrict__ a_norm,
                    int64_t T, int32_t V, int32_t S, float clip_lo, float clip_hi,
                    float* __restrict__ loss, float* __restrict__ logp_out, float* __restrict__ lse_out,
                    float* __restrict__ coef_out, float* __restrict__ entropy_out, double* block_sums, int32_t* counters,
                    const int32_t* __restrict__ seq_cnt, int agg_mode, int surrogate, int32_t global_tokens,
                    int32_t global_responses, float dual_clip, int32_t* d_status, FinalizeRange rg, OnePassFix fix) {
  // This launch covers token rows [rg.t_begin, T_end); its blocks are blocks rg.block0.. of the
  // rg.total_blocks that cover all rows (one launch, or one per chunk of the one-pass path).
  const int64_t t = rg.t_begin + (int64_t)blockIdx.x * kFinalizeThreads + threadIdx.x;
  // denominators of the expectation: this call's own counts, or the whole data-parallel batch's
  const int32_t n_tok = global_tokens > 0 ? global_tokens : counters[0];
  const int32_t s_act = global_responses > 0 ? global_responses : counters[2];
  double contrib = 0.0;
  if (t < T) {
    const int64_t tp = t - rg.t_begin;
    float m2 = -CUDART_INF_F, zt = -CUDART_INF_F;
    for (int s = 0; s < nsplit; ++s) {
      FwdPartial p = partials[(int64_t)s * rg.part_ld + tp];
      m2 = fmaxf(m2, p.m2);
      zt = fmaxf(zt, p.zt);
    }
    float l = 0.0f, ez = 0.0f;
    for (int s = 0; s < nsplit; ++s) {
      FwdPartial p = partials[(int64_t)s * rg.part_ld + tp];
      const float w = exp2f(p.m2 - m2);
      l += p.l * w;
      ez += p.pad * w;                       // sum_v e z of the split (filled when the entropy is asked for)
    }
    const float lse = (m2 + log2f(l)) * kLn2;
    if (entropy_out) entropy_out[t] = lse - ez / l;      // -sum_v p log p = lse - sum_v p z
    const int32_t yt = y[t];
    const bool on = mask ? mask[t] != 0 : true;
    float lp, coef = 0.0f;
    if (yt < 0 || yt >= V) {
      // a masked row may carry an ignore-index target (-100, -1): it takes no part in the loss
      if (on) flag(d_status, SPO_DEV_ID_OUT_OF_RANGE);
      lp = -CUDART_INF_F;
    } else {
      lp = zt - lse;
      const float ratio = expf(lp - logp_old[t]);
      int lo = 0, hi = S;                    // sequence with cu[lo] <= t < cu[lo+1]
      while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((int64_t)cu_seqlens[mid] <= t) lo = mid; else hi = mid;
      }
      const float a = a_norm[lo];
      const float hi_b = 1.0f + clip_hi, lo_b = 1.0f - clip_lo;
      const float cut = fminf(fmaxf(ratio, lo_b), hi_b);
      // per unit of token weight: the objective's term and d term / d logp
      float sur, dsur;
      if (surrogate == SPO_SUR_CISPO) {        // truncated weight, held constant, on the log-prob
        sur = cut * a * lp;
        dsur = cut * a;
      } else {                                 // PPO-Clip (a sequence-level objective fills coef later)
        sur = fminf(ratio * a, cut * a);
        bool passes = a >= 0.0f ? ratio <= hi_b : ratio >= lo_b;
        if (dual_clip > 0.0f && a < 0.0f) {    // second clip: the term may not fall below c a
          sur = fmaxf(sur, dual_clip * a);
          passes = passes && !(ratio > dual_clip);
        }
        dsur = passes ? a * ratio : 0.0f;
      }
      if (on && n_tok > 0 && surrogate != SPO_SUR_GSPO) {
        // weight of this token in the expectation: 1/n_tok, or 1/(responses * tokens of its response)
        if (agg_mode == 0) {
          contrib = (double)sur;
          if (dsur != 0.0f) coef = -dsur / (float)n_tok;
        } else {
          const float u = 1.0f / ((float)s_act * (float)seq_cnt[lo]);
          contrib = (double)sur * (double)u;
          if (dsur != 0.0f) coef = -dsur * u;
        }
      }
    }
    logp_out[t] = lp;
    lse_out[t] = lse;
    coef_out[t] = coef;
    if (fix.G) {
      // one-pass path: m2 is the row's reference exponent (common to all its partials), l the sum of
      // its stored exponentials.  A row whose logits outran the reference has l = Inf: reported, and
      // it takes no part in the gradient (its logp is -Inf, so its coef is already zero).
      if (!(l < CUDART_INF_F)) flag(d_status, SPO_DEV_NONFINITE);
      float rsc = 0.0f;
      if (coef != 0.0f && l > 0.0f && l < CUDART_INF_F) {
        rsc = -fix.grad_loss * coef / l;
        const float ey = exp2f(fmaf(zt, kLog2e, -m2));
        reinterpret_cast<__nv_bfloat16*>(fix.G)[(t - fix.g_row0) * fix.ldg + yt] = __float2bfloat16_rn(ey - l);
      }
      fix.rowscale[t] = rsc;
    }
  }
  __shared__ double s_part[kFinalizeThreads / 32];
  __shared__ int s_last;
  contrib = warp_sum_f64(contrib);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = contrib;
  __syncthreads();
  if (threadIdx.x == 0) {
    double b = 0.0;
#pragma unroll
    for (int w = 0; w < kFinalizeThreads / 32; ++w) b += s_part[w];
    block_sums[rg.block0 + blockIdx.x] = b;
    __threadfence();
    int ticket = atomicAdd(&counters[1], 1);
    s_last = (ticket == rg.total_blocks - 1);
  }
  __syncthreads();
  if (s_last) {                              // the last block to finish folds all blocks in index order
    __threadfence();
    double acc = 0.0;
    const volatile double* bs = block_sums;
    for (int i = threadIdx.x; i < rg.total_blocks; i += kFinalizeThreads) acc += bs[i];
    acc = warp_sum_f64(acc);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
#pragma unroll
      for (int w = 0; w < kFinalizeThreads / 32; ++w) tot += s_part[w];
      if (surrogate == SPO_SUR_GSPO) { /* written by the sequence-level pass */ }
      else if (n_tok <= 0) loss[0] = 0.0f;
      else loss[0] = agg_mode == 0 ? (float)(-tot / (double)n_tok) : (float)(-tot);
    }
  }
}

// One block per response: (sum mask*logp, sum mask*(logp_old - logp), sum mask).
__global__ void __launch_bounds__(256)
seq_sums_kernel(const float* __restrict__ logp, const float* __restrict__ logp_old, const uint8_t* __restrict__ mask,
                const int32_t* __restrict__ cu_seqlens, float* __restrict__ seq_sums) {
  const int s = blockIdx.x;
  const int64_t lo = cu_seqlens[s], hi = cu_seqlens[s + 1];
  double a = 0.0, b = 0.0, c = 0.0;
  for (int64_t t = lo + threadIdx.x; t < hi; t += 256) {
    if (mask && mask[t] == 0) continue;
    float lp = logp[t];
    a += lp;
    b += (double)logp_old[t] - lp;
    c += 1.0;
  }
  __shared__ double s_a[8], s_b[8], s_c[8];
  a = warp_sum_f64(a); b = warp_sum_f64(b); c = warp_sum_f64(c);
  if ((threadIdx.x & 31) == 0) { s_a[threadIdx.x >> 5] = a; s_b[threadIdx.x >> 5] = b; s_c[threadIdx.x >> 5] = c; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ta = 0, tb = 0, tc = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { ta += s_a[w]; tb += s_b[w]; tc += s_c[w]; }
    seq_sums[3 * s + 0] = (float)ta;
    seq_sums[3 * s + 1] = (float)tb;
    seq_sums[3 * s + 2] = (float)tc;
  }
}

// ---------------------------------------------------------------------------
// fp32 SIMT forward: one block per token row, one warp per vocabulary row at a time.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
fwd_f32_kernel(const float* __restrict__ H, const float* __restrict__ W, const int32_t* __restrict__ y,
               int32_t d, int32_t V, FwdPartial* __restrict__ partials) {
  extern __shared__ float s_h[];
  const int64_t t = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int k = threadIdx.x; k < d; k += 128) s_h[k] = H[t * d + k];
  __syncthreads();
  const int32_t yt = y[t];
  float m2 = -CUDART_INF_F, l = 0.0f, zt = -CUDART_INF_F, ez = 0.0f;
  for (int v = warp; v < V; v += 4) {
    const float* wr = W + (int64_t)v * d;
    float acc = 0.0f;
    for (int k = lane; k < d; k += 32) acc = fmaf(wr[k], s_h[k], acc);
    const float z = warp_sum_f32(acc);
    const float z2 = z * kLog2e;
    const float mn = fmaxf(m2, z2);
    const float down = exp2f(m2 - mn), e = exp2f(z2 - mn);
    l = l * down + e;
    ez = ez * down + e * z;
    m2 = mn;
    if (v == yt) zt = z;
  }
  __shared__ float s_m[4], s_l[4], s_z[4], s_e[4];
  if (lane == 0) { s_m[warp] = m2; s_l[warp] = l; s_z[warp] = zt; s_e[warp] = ez; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float mm = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
    float ll = 0.0f, zz = -CUDART_INF_F, ee = 0.0f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      if (s_l[w] > 0.0f) { ll += s_l[w] * exp2f(s_m[w] - mm); ee += s_e[w] * exp2f(s_m[w] - mm); }
      zz = fmaxf(zz, s_z[w]);
    }
    FwdPartial p;
    p.m2 = mm; p.l = ll; p.zt = zz; p.pad = ee;
    partials[t] = p;
  }
}

// ---------------------------------------------------------------------------
// fp32 SIMT backward.  One block per output row x (a token row of dH, or a vocabulary
// row of dW).  For every row j of the other matrix Y: s = <x, Y_j>, g = c*(1[v=y_t] - e^{s-lse_t}),
// out += g * Y_j.  DW = false: x = H[t], Y = W.  DW = true: x = W[v], Y = H.
// ---------------------------------------------------------------------------
constexpr int kBwdChunk = 256;
constexpr int kBwdMaxPerThread = 32;       // d <= 128 * 32

template <bool DW>
__global__ void __launch_bounds__(128)
bwd_f32_kernel(const float* __restrict__ H, const float* __restrict__ W, const int32_t* __restrict__ y,
               const float* __restrict__ lse, const float* __restrict__ coef, float grad_loss,
               int64_t T, int32_t d, int32_t V, void* out, int out_bf16, int accumulate) {
  extern __shared__ float s_mem[];
  float* s_x = s_mem;                       // [d]
  float* s_g = s_mem + d;                   // [kBwdChunk]
  const int64_t row = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* X = DW ? W : H;
  const float* Y = DW ? H : W;
  const int64_t n_other = DW ? T : (int64_t)V;
  for (int k = threadIdx.x; k < d; k += 128) s_x[k] = X[row * d + k];
  float acc[kBwdMaxPerThread];
#pragma unroll
  for (int i = 0; i < kBwdMaxPerThread; ++i) acc[i] = 0.0f;
  float c_row = 0.0f, lse_row = 0.0f;
  int32_t y_row = -1;
  if (!DW) { c_row = grad_loss * coef[row]; lse_row = lse[row]; y_row = y[row]; }
  __syncthreads();
  for (int64_t j0 = 0; j0 < n_other; j0 += kBwdChunk) {
    const int n_here = (int)((n_other - j0) < kBwdChunk ? (n_other - j0) : kBwdChunk);
    for (int jj = warp; jj < n_here; jj += 4) {
      const int64_t j = j0 + jj;
      float c = c_row, ls = lse_row;
      bool hit;
      if (DW) { c = grad_loss * coef[j]; ls = lse[j]; hit = (y[j] == (int32_t)row); }
      else    { hit = ((int32_t)j == y_row); }
      float g = 0.0f;
      if (c != 0.0f) {                      // warp-uniform
        const float* yr = Y + j * d;
        float a = 0.0f;
        for (int k = lane; k < d; k += 32) a = fmaf(yr[k], s_x[k], a);
        const float s = warp_sum_f32(a);
        g = c * ((hit ? 1.0f : 0.0f) - expf(s - ls));
      }
      if (lane == 0) s_g[jj] = g;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kBwdMaxPerThread; ++i) {
      const int k = threadIdx.x + 128 * i;
      if (k < d) {
        float a = acc[i];
        for (int jj = 0; jj < n_here; ++jj) a = fmaf(s_g[jj], Y[(j0 + jj) * d + k], a);
        acc[i] = a;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < kBwdMaxPerThread; ++i) {
    const int k = threadIdx.x + 128 * i;
    if (k < d) {
      const int64_t o = row * d + k;
      if (out_bf16) {
        reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(acc[i]);
      } else {
        float* of = reinterpret_cast<float*>(out);
        of[o] = accumulate ? of[o] + acc[i] : acc[i];
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Row compaction for the backward: tokens whose coef is zero (masked, or clipped on the side
// that stops the gradient) contribute nothing to dH or dW.
// ---------------------------------------------------------------------------
constexpr int kRowsPerBlock = 1024;

// A row is listed when its coef is non-zero (coef given) or when its mask byte is non-zero (mask given).
__device__ __forceinline__ int row_is_listed(const float* coef, const uint8_t* mask, int64_t t) {
  return coef ? (coef[t] != 0.0f) : (mask[t] != 0);
}

__global__ void __launch_bounds__(1024)
active_count_kernel(const float* __restrict__ coef, const uint8_t* __restrict__ mask, int64_t T,
                    int32_t* __restrict__ block_cnt) {
  const int64_t t = (int64_t)blockIdx.x * kRowsPerBlock + threadIdx.x;
  const int on = (t < T && row_is_listed(coef, mask, t)) ? 1 : 0;
  const int total = __syncthreads_count(on);
  if (threadIdx.x == 0) block_cnt[blockIdx.x] = total;
}

// Exclusive scan of the block counts by one block; *d_count = number of active rows.
__global__ void __launch_bounds__(1024)
active_scan_kernel(int32_t* block_cnt, int64_t n_blocks, int32_t* __restrict__ d_count) {
  __shared__ int s_warp[32];
  __shared__ int s_run;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_run = 0;
  __syncthreads();
  for (int64_t b0 = 0; b0 < n_blocks; b0 += 1024) {
    const int64_t b = b0 + tid;
    const int v = b < n_blocks ? block_cnt[b] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += x;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = s_run;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    if (b < n_blocks) block_cnt[b] = before + incl - v;
    __syncthreads();
    if (tid == 1023) s_run = before + incl;
    __syncthreads();
  }
  if (tid == 0) *d_count = s_run;
}

__global__ void __launch_bounds__(1024)
active_write_kernel(const float* __restrict__ coef, const uint8_t* __restrict__ mask, int64_t T,
                    const int32_t* __restrict__ block_off, int32_t* __restrict__ rows) {
  __shared__ int s_warp[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t t = (int64_t)blockIdx.x * kRowsPerBlock + tid;
  const int on = (t < T && row_is_listed(coef, mask, t)) ? 1 : 0;
  const unsigned bal = __ballot_sync(0xffffffffu, on);
  if (lane == 0) s_warp[warp] = __popc(bal);
  __syncthreads();
  int before = block_off[blockIdx.x];
  for (int w = 0; w < warp; ++w) before += s_warp[w];
  if (on) rows[before + __popc(bal & ((1u << lane) - 1))] = (int32_t)t;
}

// One warp per active row: copy the row of H (16-byte pieces) and its per-token scalars.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ H, const int32_t* __restrict__ y, const float* __restrict__ lse,
                   const float* __restrict__ coef, const int32_t* __restrict__ rows, int64_t n_act, int64_t T,
                   int row_vec, uint4* __restrict__ H_act, int32_t* __restrict__ y_act, float* __restrict__ lse_act,
                   float* __restrict__ coef_act, int32_t* d_status) {
  const int lane = threadIdx.x & 31;
  for (int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5; i < n_act; i += ((int64_t)gridDim.x * 256) >> 5) {
    const int64_t t = rows[i];
    if (t < 0 || t >= T) {                  // a row index outside the batch: reported, never dereferenced
      if (lane == 0) { flag(d_status, SPO_DEV_ID_OUT_OF_RANGE); y_act[i] = 0; lse_act[i] = 0.0f; coef_act[i] = 0.0f; }
      for (int k = lane; k < row_vec; k += 32) H_act[i * row_vec + k] = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
    for (int k = lane; k < row_vec; k += 32) H_act[i * row_vec + k] = __ldg(H + t * row_vec + k);
    if (lane == 0) { y_act[i] = y[t]; lse_act[i] = lse[t]; coef_act[i] = coef[t]; }
  }
}

__global__ void __launch_bounds__(256)
scatter_rows_kernel(const uint4* __restrict__ dH_act, const int32_t* __restrict__ rows, int64_t n_act, int64_t T,
                    int row_vec, uint4* __restrict__ dH) {
  const int lane = threadIdx.x & 31;
  for (int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5; i < n_act; i += ((int64_t)gridDim.x * 256) >> 5) {
    const int64_t t = rows[i];
    if (t < 0 || t >= T) continue;          // reported by the gather of the same list
    for (int k = lane; k < row_vec; k += 32) dH[t * row_vec + k] = dH_act[i * row_vec + k];
  }
}


// One warp per row: out[i] = rowscale[t0 + i] * H[t0 + i], bf16, 16-byte pieces.
__global__ void __launch_bounds__(256)
scale_rows_kernel(const uint4* __restrict__ H, const float* __restrict__ rowscale, int64_t t0, int64_t rows,
                  int row_vec, uint4* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  for (int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5; i < rows; i += ((int64_t)gridDim.x * 256) >> 5) {
    const float rs = rowscale[t0 + i];
    const uint4* src = H + (t0 + i) * row_vec;
    uint4* dst = out + i * row_vec;
    for (int k = lane; k < row_vec; k += 32) {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (rs != 0.0f) {
        const uint4 h = __ldg(src + k);
        const uint32_t w[4] = {h.x, h.y, h.z, h.w};
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __nv_bfloat162 pr2 = __floats2bfloat162_rn(__uint_as_float(w[q] << 16) * rs,
                                                           __uint_as_float(w[q] & 0xFFFF0000u) * rs);
          o[q] = *reinterpret_cast<const uint32_t*>(&pr2);
        }
        v = make_uint4(o[0], o[1], o[2], o[3]);
      }
      dst[k] = v;
    }
  }
}

// dW added, row by row, into the shards that own its vocabulary rows (the reduce-scatter form of the
// paths whose last contraction does not do it itself).  16-byte pieces, vector store-reductions.
struct ShardTable { float* shard[SPO_MAX_DW_SHARDS]; int n; int64_t rows; };

__global__ void __launch_bounds__(256)
dw_scatter_add_kernel(const float4* __restrict__ dW, int64_t n_vec, int row_vec, ShardTable tb) {
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * 256) {
    const int64_t v = i / row_vec;
    const int owner = (int)(v / tb.rows);
    const float4 x = dW[i];
    float* dst = tb.shard[owner] + ((v - (int64_t)owner * tb.rows) * row_vec + (i - v * row_vec)) * 4;
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w)
                 : "memory");
  }
}

// Sequence-level objective, one block per response: r = exp(mean over its unmasked tokens of
// logp - logp_old), term = min(r a, clip(r) a), and the coef all its unmasked tokens share.
__global__ void __launch_bounds__(256)
seq_level_terms_kernel(const float* __restrict__ logp, const float* __restrict__ logp_old,
                       const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu_seqlens,
                       const float* __restrict__ a_norm, float clip_lo, float clip_hi,
                       const int32_t* __restrict__ counters, int32_t global_responses, float dual_clip,
                       float* __restrict__ seq_coef, double* __restrict__ seq_term) {
  const int s = blockIdx.x;
  const int64_t lo = cu_seqlens[s], hi = cu_seqlens[s + 1];
  double sum = 0.0, cnt = 0.0;
  for (int64_t t = lo + threadIdx.x; t < hi; t += 256) {
    if (mask && mask[t] == 0) continue;
    sum += (double)logp[t] - (double)logp_old[t];
    cnt += 1.0;
  }
  __shared__ double s_a[8], s_c[8];
  sum = warp_sum_f64(sum); cnt = warp_sum_f64(cnt);
  if ((threadIdx.x & 31) == 0) { s_a[threadIdx.x >> 5] = sum; s_c[threadIdx.x >> 5] = cnt; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ts = 0, tc = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { ts += s_a[w]; tc += s_c[w]; }
    const int32_t s_act = global_responses > 0 ? global_responses : counters[2];
    float c = 0.0f;
    double term = 0.0;
    if (tc > 0.0 && s_act > 0) {
      const double r = exp(ts / tc);
      const double a = (double)a_norm[s];
      const double hi_b = 1.0 + (double)clip_hi, lo_b = 1.0 - (double)clip_lo;
      term = fmin(r * a, fmin(fmax(r, lo_b), hi_b) * a);
      bool passes = a >= 0.0 ? r <= hi_b : r >= lo_b;
      if (dual_clip > 0.0f && a < 0.0) {
        term = fmax(term, (double)dual_clip * a);
        passes = passes && !(r > (double)dual_clip);
      }
      if (passes) c = (float)(-a * r / ((double)s_act * tc));
    }
    seq_coef[s] = c;
    seq_term[s] = term;
  }
}

// coef of every token from its response's value; block 0 also folds the responses' terms (index
// order, fixed tree) into the loss.
__global__ void __launch_bounds__(256)
seq_level_apply_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu_seqlens, int64_t T, int32_t S,
                       const float* __restrict__ seq_coef, const double* __restrict__ seq_term,
                       const int32_t* __restrict__ counters, int32_t global_responses, float* __restrict__ coef,
                       float* __restrict__ loss) {
  const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (t < T) {
    int lo = 0, hi = S;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if ((int64_t)cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    const bool on = mask ? mask[t] != 0 : true;
    coef[t] = on ? seq_coef[lo] : 0.0f;
  }
  if (blockIdx.x == 0) {
    __shared__ double s_part[8];
    double acc = 0.0;
    for (int i = threadIdx.x; i < S; i += 256) acc += seq_term[i];
    acc = warp_sum_f64(acc);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = 0.0;
#pragma unroll
      for (int w = 0; w < 8; ++w) tot += s_part[w];
      const int32_t s_act = global_responses > 0 ? global_responses : counters[2];
      loss[0] = s_act > 0 ? (float)(-tot / (double)s_act) : 0.0f;
    }
  }
}

// Diagnostics of the policy update over the unmasked tokens, one block (fixed reduction order):
// count, mean ratio, share of tokens whose gradient the clip stops, two sampled KL estimates,
// largest / smallest ratio, share of ratios outside the clip bounds.
__global__ void __launch_bounds__(1024)
loss_stats_kernel(const float* __restrict__ logp, const float* __restrict__ logp_old, const uint8_t* __restrict__ mask,
                  const int32_t* __restrict__ cu_seqlens, const float* __restrict__ a_norm, int64_t T, int32_t S,
                  float clip_lo, float clip_hi, float dual_clip, float* __restrict__ out) {
  const float hi_b = 1.0f + clip_hi, lo_b = 1.0f - clip_lo;
  double acc[6] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0};     // count, ratio, stopped, -d, k3, outside
  float rmax = -CUDART_INF_F, rmin = CUDART_INF_F;
  for (int64_t t = threadIdx.x; t < T; t += 1024) {
    if (mask && mask[t] == 0) continue;
    int lo = 0, hi = S;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if ((int64_t)cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    const float a = a_norm[lo];
    const float d = logp[t] - logp_old[t];
    const float r = expf(d);
    const bool stopped = a > 0.0f ? r > hi_b : (a < 0.0f ? (r < lo_b || (dual_clip > 0.0f && r > dual_clip)) : false);
    acc[0] += 1.0;
    acc[1] += (double)r;
    acc[2] += stopped ? 1.0 : 0.0;
    acc[3] -= (double)d;
    acc[4] += (double)r - 1.0 - (double)d;
    acc[5] += (r > hi_b || r < lo_b) ? 1.0 : 0.0;
    rmax = fmaxf(rmax, r);
    rmin = fminf(rmin, r);
  }
  __shared__ double s_acc[32][6];
  __shared__ float s_max[32], s_min[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < 6; ++k) acc[k] = warp_sum_f64(acc[k]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
    rmin = fminf(rmin, __shfl_xor_sync(0xffffffffu, rmin, o));
  }
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < 6; ++k) s_acc[warp][k] = acc[k];
    s_max[warp] = rmax; s_min[warp] = rmin;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot[6] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
    float mx = -CUDART_INF_F, mn = CUDART_INF_F;
    for (int w = 0; w < 32; ++w) {
#pragma unroll
      for (int k = 0; k < 6; ++k) tot[k] += s_acc[w][k];
      mx = fmaxf(mx, s_max[w]); mn = fminf(mn, s_min[w]);
    }
    if (tot[0] > 0.0) {
      out[0] = (float)tot[0];
      out[1] = (float)(tot[1] / tot[0]);
      out[2] = (float)(tot[2] / tot[0]);
      out[3] = (float)(tot[3] / tot[0]);
      out[4] = (float)(tot[4] / tot[0]);
      out[5] = mx;
      out[6] = mn;
      out[7] = (float)(tot[5] / tot[0]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) out[k] = 0.0f;
    }
  }
}

// Sequence boundaries of the compacted batch: cu_act[s] = number of listed rows below cu_seqlens[s]
// (rows is ascending, so a lower bound).
__global__ void __launch_bounds__(256)
compact_cu_seqlens_kernel(const int32_t* __restrict__ rows, int64_t n_act, const int32_t* __restrict__ cu_seqlens,
                          int32_t S, int32_t* __restrict__ cu_act) {
  const int s = blockIdx.x * 256 + threadIdx.x;
  if (s > S) return;
  const int32_t bound = cu_seqlens[s];
  int64_t lo = 0, hi = n_act;                 // first i with rows[i] >= bound
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (rows[mid] < bound) lo = mid + 1; else hi = mid;
  }
  cu_act[s] = (int32_t)lo;
}

// logp / lse / coef of the compacted rows back to their places in the full arrays.
__global__ void __launch_bounds__(256)
scatter_scalars_kernel(const float* __restrict__ logp_act, const float* __restrict__ lse_act,
                       const float* __restrict__ coef_act, const int32_t* __restrict__ rows, int64_t n_act, int64_t T,
                       float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ coef) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n_act) return;
  const int64_t t = rows[i];
  if (t < 0 || t >= T) return;              // reported by the gather of the same list
  logp[t] = logp_act[i];
  lse[t] = lse_act[i];
  coef[t] = coef_act[i];
}

}  // namespace

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------

cudaError_t launch_fwd_prepare(const uint8_t* mask, int64_t T, const int32_t* cu_seqlens, int32_t S,
                               int need_seq_counts, int32_t* seq_cnt, int32_t* counters, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(counters, 0, 4 * sizeof(int32_t), st);
  if (e != cudaSuccess) return e;
  if (need_seq_counts && S > 0 && T > 0) {
    seq_count_kernel<<<S, 256, 0, st>>>(mask, cu_seqlens, seq_cnt, counters);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (mask) {
    int64_t blocks = ceil_div(T > 0 ? T : 1, 256 * 8);
    int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    count_mask_kernel<<<(unsigned)blocks, 256, 0, st>>>(mask, T, counters);
  } else {
    set_count_kernel<<<1, 1, 0, st>>>((int32_t)T, counters);
  }
  return cudaGetLastError();
}

cudaError_t launch_fwd_finalize(const FwdPartial* partials, int nsplit, const int32_t* y,
                                const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                                const float* a_norm, int64_t T, int32_t V, int32_t S,
                                float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                                double* block_sums, int32_t* counters, const int32_t* seq_cnt, const spo_params& pr,
                                int64_t fin_blocks, int32_t* d_status, cudaStream_t st,
                                const FinalizeRange* range, const OnePassFix* fix) {
  // Default: one launch over all rows.  With a range: rows [t_begin, T) of a larger batch whose
  // blocks are numbered from block0; T is then the end of the range and the per-response sums
  // are left to the launch that covers the last rows.
  FinalizeRange rg;
  rg.t_begin = 0; rg.part_ld = T; rg.block0 = 0; rg.total_blocks = (int)fin_blocks; rg.last = 1;
  unsigned blocks = (unsigned)fin_blocks;
  if (range) {
    rg = *range;
    blocks = (unsigned)ceil_div(T - rg.t_begin, kFinalizeThreads);
  }
  if (blocks == 0) return cudaSuccess;
  fwd_finalize_kernel<<<blocks, kFinalizeThreads, 0, st>>>(
      partials, nsplit, y, logp_old, mask, cu_seqlens, a_norm, T, V, S, pr.clip_lo, pr.clip_hi,
      loss, logp, lse, coef, entropy, block_sums, counters, seq_cnt, pr.agg_mode, pr.surrogate, pr.global_tokens,
      pr.global_responses, pr.dual_clip, d_status, rg, fix ? *fix : OnePassFix{nullptr, 0, 0, nullptr, 0.0f});
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (seq_sums && S > 0 && rg.last) {
    seq_sums_kernel<<<S, 256, 0, st>>>(logp, logp_old, mask, cu_seqlens, seq_sums);
    e = cudaGetLastError();
  }
  return e;
}

cudaError_t launch_seq_level_objective(const float* logp, const float* logp_old, const uint8_t* mask,
                                       const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t S,
                                       const spo_params& pr, const int32_t* counters,
                                       float* seq_coef, double* seq_term, float* coef, float* loss, cudaStream_t st) {
  const int32_t global_responses = pr.global_responses;
  if (S > 0) {
    seq_level_terms_kernel<<<S, 256, 0, st>>>(logp, logp_old, mask, cu_seqlens, a_norm, pr.clip_lo, pr.clip_hi, counters,
                                              global_responses, pr.dual_clip, seq_coef, seq_term);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  seq_level_apply_kernel<<<(unsigned)ceil_div(T > 0 ? T : 1, 256), 256, 0, st>>>(
      mask, cu_seqlens, T, S, seq_coef, seq_term, counters, global_responses, coef, loss);
  return cudaGetLastError();
}

cudaError_t launch_fwd_f32(const float* H, const float* W, const int32_t* y, int64_t T, int32_t d, int32_t V,
                           FwdPartial* partials, cudaStream_t st) {
  if (T == 0) return cudaSuccess;
  fwd_f32_kernel<<<(unsigned)T, 128, sizeof(float) * d, st>>>(H, W, y, d, V, partials);
  return cudaGetLastError();
}

cudaError_t launch_bwd_f32(const float* H, const float* W, const int32_t* y, const float* lse,
                           const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V,
                           void* dH, int32_t dH_dtype, float* dW, int accumulate, cudaStream_t st) {
  const size_t smem = sizeof(float) * (d + kBwdChunk);
  if (T > 0) {
    bwd_f32_kernel<false><<<(unsigned)T, 128, smem, st>>>(H, W, y, lse, coef, grad_loss, T, d, V, dH,
                                                          dH_dtype == SPO_DTYPE_BF16, 0);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  bwd_f32_kernel<true><<<(unsigned)V, 128, smem, st>>>(H, W, y, lse, coef, grad_loss, T, d, V, dW, 0, accumulate);
  return cudaGetLastError();
}

cudaError_t launch_active_rows(const float* coef, const uint8_t* mask, int64_t T, int32_t* rows, int32_t* d_count,
                               int32_t* block_cnt, cudaStream_t st) {
  const int64_t n_blocks = ceil_div(T > 0 ? T : 1, kRowsPerBlock);
  active_count_kernel<<<(unsigned)n_blocks, 1024, 0, st>>>(coef, mask, T, block_cnt);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  active_scan_kernel<<<1, 1024, 0, st>>>(block_cnt, n_blocks, d_count);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  active_write_kernel<<<(unsigned)n_blocks, 1024, 0, st>>>(coef, mask, T, block_cnt, rows);
  return cudaGetLastError();
}

size_t active_rows_ws_bytes(int64_t T) {
  return align_up(sizeof(int32_t) * (size_t)ceil_div(T > 0 ? T : 1, kRowsPerBlock), 256);
}

cudaError_t launch_gather_rows(const void* H, const int32_t* y, const float* lse, const float* coef,
                               const int32_t* rows, int64_t n_act, int64_t T, int32_t row_bytes, void* H_act,
                               int32_t* y_act, float* lse_act, float* coef_act, int32_t* d_status, cudaStream_t st) {
  if (n_act == 0) return cudaSuccess;
  int64_t blocks = ceil_div(n_act * 32, 256);
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  gather_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(H), y, lse, coef, rows, n_act, T,
                                                       row_bytes / 16, reinterpret_cast<uint4*>(H_act), y_act, lse_act,
                                                       coef_act, d_status);
  return cudaGetLastError();
}

cudaError_t launch_scale_rows(const void* H, const float* rowscale, int64_t t0, int64_t rows, int32_t row_bytes,
                              void* out, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  int64_t blocks = ceil_div(rows * 32, 256);
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  scale_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(H), rowscale, t0, rows,
                                                      row_bytes / 16, reinterpret_cast<uint4*>(out));
  return cudaGetLastError();
}

cudaError_t launch_dw_scatter_add(const float* dW, int32_t V, int32_t d, const spo_dw_shards& sh, cudaStream_t st) {
  ShardTable tb{};
  tb.n = sh.n_shards;
  tb.rows = sh.rows_per_shard;
  for (int k = 0; k < sh.n_shards; ++k) tb.shard[k] = sh.shard[k];
  const int64_t n_vec = (int64_t)V * d / 4;
  int64_t blocks = ceil_div(n_vec, 256 * 4);
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  dw_scatter_add_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(dW), n_vec, d / 4, tb);
  return cudaGetLastError();
}

cudaError_t launch_loss_stats(const float* logp, const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                              const float* a_norm, int64_t T, int32_t S, const spo_params& pr, float* out,
                              cudaStream_t st) {
  loss_stats_kernel<<<1, 1024, 0, st>>>(logp, logp_old, mask, cu_seqlens, a_norm, T, S, pr.clip_lo, pr.clip_hi,
                                        pr.dual_clip, out);
  return cudaGetLastError();
}

cudaError_t launch_compact_cu_seqlens(const int32_t* rows, int64_t n_act, const int32_t* cu_seqlens, int32_t S,
                                      int32_t* cu_act, cudaStream_t st) {
  compact_cu_seqlens_kernel<<<(unsigned)ceil_div(S + 1, 256), 256, 0, st>>>(rows, n_act, cu_seqlens, S, cu_act);
  return cudaGetLastError();
}

cudaError_t launch_scatter_scalars(const float* logp_act, const float* lse_act, const float* coef_act,
                                   const int32_t* rows, int64_t n_act, int64_t T, float* logp, float* lse, float* coef,
                                   cudaStream_t st) {
  if (n_act == 0) return cudaSuccess;
  scatter_scalars_kernel<<<(unsigned)ceil_div(n_act, 256), 256, 0, st>>>(logp_act, lse_act, coef_act, rows, n_act, T,
                                                                        logp, lse, coef);
  return cudaGetLastError();
}

cudaError_t launch_scatter_rows(const void* dH_act, const int32_t* rows, int64_t n_act, int64_t T, int32_t row_bytes,
                                void* dH, cudaStream_t st) {
  if (n_act == 0) return cudaSuccess;
  int64_t blocks = ceil_div(n_act * 32, 256);
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  scatter_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(dH_act), rows, n_act, T,
                                                        row_bytes / 16, reinterpret_cast<uint4*>(dH));
  return cudaGetLastError();
}

}  // namespace spo
