// C-ABI entry points of libspo: argument checks, workspace carving, dispatch.
// See include/spo.h for the contract of every call.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "spo_internal.h"

namespace spo {

static thread_local int32_t g_last_cuda_error = 0;

int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
  if (dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      return 148;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

int device_is_sm100() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return major == 10;
}

int fwd_bf16_nsplit(int64_t T, int32_t d, int32_t V);   // spo_loss_tc.cu

FwdWs fwd_ws_layout(int64_t T, int32_t d, int32_t V, int32_t dtype, int32_t S) {
  FwdWs L{};
  L.nsplit = dtype == SPO_DTYPE_BF16 ? fwd_bf16_nsplit(T, d, V) : 1;
  L.fin_blocks = ceil_div(T > 0 ? T : 1, kFinalizeThreads);
  size_t off = 0;
  L.progress = off;   off = align_up(off + kProgressBytes, 256);
  L.partials = off;   off = align_up(off + sizeof(FwdPartial) * (size_t)L.nsplit * (size_t)(T > 0 ? T : 1), 256);
  L.block_sums = off; off = align_up(off + sizeof(double) * (size_t)L.fin_blocks, 256);
  L.counters = off;   off = align_up(off + 4 * sizeof(int32_t), 256);
  L.seq_cnt = off;    off = align_up(off + sizeof(int32_t) * (size_t)(S > 0 ? S : 1), 256);
  L.seq_coef = off;   off = align_up(off + sizeof(float) * (size_t)(S > 0 ? S : 1), 256);
  L.seq_term = off;   off = align_up(off + sizeof(double) * (size_t)(S > 0 ? S : 1), 256);
  L.total = off;
  return L;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int32_t record_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int32_t)e;
  return SPO_ERR_CUDA;
}
static inline int32_t cuda_fail(cudaError_t e) { return record_cuda_error(e); }

static bool params_ok(const spo_params* p) {
  if (!p) return false;
  if (!(p->rho_min >= 0.0f) || !(p->rho_max <= 1.0f) || !(p->rho_min <= p->rho_max)) return false;
  if (!(p->d_half > 0.0f)) return false;
  if (!(p->eps_explore >= 0.0f)) return false;
  if (!(p->clip_lo >= 0.0f) || !(p->clip_lo < 1.0f) || !(p->clip_hi >= 0.0f)) return false;
  if (!(p->norm_eps >= 0.0f)) return false;
  if (p->norm_ddof != 0 && p->norm_ddof != 1) return false;
  if (p->agg_mode != SPO_AGG_TOKEN_MEAN && p->agg_mode != SPO_AGG_SEQ_MEAN) return false;
  if (p->global_tokens < 0 || p->global_responses < 0) return false;
  if (p->surrogate != SPO_SUR_PPO_CLIP && p->surrogate != SPO_SUR_CISPO && p->surrogate != SPO_SUR_GSPO) return false;
  if (!(p->dual_clip == 0.0f || (p->dual_clip > 1.0f && p->dual_clip < 3.0e38f))) return false;
  if (!(p->near_zero_tau_lo >= 0.0f) || !(p->near_zero_tau_hi >= 0.0f)) return false;
  return true;
}

}  // namespace spo

namespace spo {

// The launches of spo_loss_fwd: token count, logits contraction into per-split partials, per-token
// finalisation, and for the sequence-level objective the pass that needs every token's logp first.
static cudaError_t forward_launches(const void* H, const void* W, int32_t dtype, const int32_t* y,
                                    const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                                    const float* a_norm, int64_t T, int32_t d, int32_t V, int32_t S, float* loss,
                                    float* logp, float* lse, float* coef, float* seq_sums, float* entropy, char* w8,
                                    const FwdWs& L,
                                    const spo_params* params, int32_t* d_status, cudaStream_t st) {
  FwdPartial* partials = reinterpret_cast<FwdPartial*>(w8 + L.partials);
  double* block_sums = reinterpret_cast<double*>(w8 + L.block_sums);
  int32_t* counters = reinterpret_cast<int32_t*>(w8 + L.counters);
  int32_t* seq_cnt = reinterpret_cast<int32_t*>(w8 + L.seq_cnt);
  const bool seq_level = params->surrogate == SPO_SUR_GSPO;
  cudaError_t e = launch_fwd_prepare(mask, T, cu_seqlens, S, params->agg_mode != 0 || seq_level, seq_cnt, counters, st);
  if (e != cudaSuccess) return e;
  if (dtype == SPO_DTYPE_BF16)
    e = launch_fwd_bf16(H, W, y, T, d, V, partials, L.nsplit, entropy != nullptr,
                        reinterpret_cast<uint32_t*>(w8 + L.progress), d_status, st);
  else
    e = launch_fwd_f32((const float*)H, (const float*)W, y, T, d, V, partials, st);
  if (e != cudaSuccess) return e;
  e = launch_fwd_finalize(partials, L.nsplit, y, logp_old, mask, cu_seqlens, a_norm, T, V, S, loss, logp, lse, coef,
                          seq_sums, entropy, block_sums, counters, seq_cnt, *params, L.fin_blocks, d_status, st);
  if (e != cudaSuccess || !seq_level) return e;
  return launch_seq_level_objective(logp, logp_old, mask, cu_seqlens, a_norm, T, S, *params, counters,
                                    reinterpret_cast<float*>(w8 + L.seq_coef),
                                    reinterpret_cast<double*>(w8 + L.seq_term), coef, loss, st);
}

}  // namespace spo

using namespace spo;

extern "C" {

int32_t spo_default_params(spo_params* p) {
  if (!p) return SPO_ERR_INVALID_ARG;
  p->rho_min = 0.875f;
  p->rho_max = 0.96f;
  p->d_half = 0.1f;
  p->eps_explore = 0.05f;
  p->clip_lo = 0.2f;
  p->clip_hi = 0.28f;
  p->norm_eps = 1e-8f;
  p->norm_ddof = 0;
  p->agg_mode = SPO_AGG_TOKEN_MEAN;
  p->global_tokens = 0;
  p->global_responses = 0;
  p->surrogate = SPO_SUR_PPO_CLIP;
  p->dual_clip = 0.0f;
  p->near_zero_tau_lo = 1e-4f;
  p->near_zero_tau_hi = 0.02f;
  return SPO_OK;
}

int32_t spo_tracker_init(float* ab, const float* v0, int64_t N, const spo_params* params, void* stream) {
  if (!params_ok(params) || N < 0 || (N > 0 && (!ab || !v0))) return SPO_ERR_INVALID_ARG;
  if (!(params->rho_min < 1.0f)) return SPO_ERR_INVALID_ARG;
  if (N >= ((int64_t)1 << 31)) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(v0)) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const float n0 = 1.0f / (1.0f - params->rho_min);
  cudaError_t e = launch_tracker_init(ab, v0, N, n0, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_sample_prompts(const float* ab, int64_t N, const float* uniforms, int32_t M, int32_t B,
                           int32_t* out_ids, float* out_w, void* ws, size_t ws_bytes,
                           const spo_params* params, int32_t* d_status, void* stream) {
  if (!params_ok(params) || !ab || !uniforms || !out_ids || !ws) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31) || B < 1 || M < B || M > (1 << 20)) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(uniforms) || !aligned16(out_ids) || !aligned16(out_w) || !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const SampleWs L = sample_ws_layout(N, M);
  if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = launch_sample(ab, N, uniforms, M, B, out_ids, out_w, (char*)ws, L, params->eps_explore, d_status,
                                (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_advantages(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                       float* a_raw, float* a_norm, float* stats, void* ws, size_t ws_bytes,
                       const spo_params* params, int32_t* d_status, void* stream) {
  if (!params_ok(params) || !ab || !ids || !r || !a_norm) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31) || B < 1) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(ids) || !aligned16(r) || !aligned16(a_raw) || !aligned16(a_norm) ||
      !aligned16(stats) || !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  if (B > kAdvSingleBlockMax) {
    if (!ws) return SPO_ERR_INVALID_ARG;
    if (ws_bytes < spo_workspace_bytes(SPO_WS_ADVANTAGES, 0, 0, 0, N, B, 0)) return SPO_ERR_WORKSPACE_TOO_SMALL;
  }
  cudaError_t e = launch_advantages(const_cast<float*>(ab), N, ids, r, B, a_raw, a_norm, stats, ws, *params, nullptr,
                                    false, d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_advantages_update(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                              int32_t kl_is_table, int32_t B, float* a_raw, float* a_norm, float* stats, void* ws,
                              size_t ws_bytes, const spo_params* params, int32_t* d_status, void* stream) {
  if (!params_ok(params) || !ab || !ids || !r || !kl || !a_norm) return SPO_ERR_INVALID_ARG;
  if (kl_is_table != 0 && kl_is_table != 1) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31) || B < 1) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(ids) || !aligned16(r) || !aligned16(kl) || !aligned16(a_raw) ||
      !aligned16(a_norm) || !aligned16(stats) || !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  if (B > kAdvSingleBlockMax) {
    if (!ws) return SPO_ERR_INVALID_ARG;
    if (ws_bytes < spo_workspace_bytes(SPO_WS_ADVANTAGES, 0, 0, 0, N, B, 0)) return SPO_ERR_WORKSPACE_TOO_SMALL;
  }
  const AdvUpdate upd = {kl, kl_is_table};
  cudaError_t e = launch_advantages(ab, N, ids, r, B, a_raw, a_norm, stats, ws, *params, &upd, false, d_status,
                                    (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_advantages_apply(const float* a_raw, int32_t B, float mu, float sigma, float* a_norm,
                             const spo_params* params, void* stream) {
  if (!params_ok(params) || B < 0 || (B > 0 && (!a_raw || !a_norm))) return SPO_ERR_INVALID_ARG;
  if (!(sigma >= 0.0f) || !(mu == mu)) return SPO_ERR_INVALID_ARG;
  if (!aligned16(a_raw) || !aligned16(a_norm)) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaError_t e = launch_advantages_apply(a_raw, B, mu, sigma, params->norm_eps, a_norm, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_tracker_update(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                           int32_t kl_is_table, int32_t B, const spo_params* params, int32_t* d_status,
                           void* stream) {
  if (!params_ok(params) || !ab || B < 0 || (B > 0 && (!ids || !r || !kl))) return SPO_ERR_INVALID_ARG;
  if (kl_is_table != 0 && kl_is_table != 1) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31)) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(ids) || !aligned16(r) || !aligned16(kl)) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaError_t e = launch_tracker_update(ab, N, ids, r, kl, kl_is_table, B, params->rho_min, params->rho_max,
                                        params->d_half, d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_tracker_update_repeats(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                                   int32_t kl_is_table, int32_t B, void* ws, size_t ws_bytes,
                                   const spo_params* params, int32_t* d_status, void* stream) {
  if (!params_ok(params) || !ab || B < 0 || (B > 0 && (!ids || !r || !kl || !ws))) return SPO_ERR_INVALID_ARG;
  if (kl_is_table != 0 && kl_is_table != 1) return SPO_ERR_INVALID_ARG;
  if (N < 1 || N >= ((int64_t)1 << 31) || B > kRepeatsMaxBatch) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(ab) || !aligned16(ids) || !aligned16(r) || !aligned16(kl) || !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const RepeatsWs L = repeats_ws_layout(B);
  if (B > 0 && ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = launch_tracker_update_repeats(ab, N, ids, r, kl, kl_is_table, B, (char*)ws, L, params->rho_min,
                                                params->rho_max, params->d_half, d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

static int32_t check_loss_shape(int32_t dtype, int64_t T, int32_t d, int32_t V) {
  if (dtype != SPO_DTYPE_F32 && dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (T < 0 || d < 1 || V < 1) return SPO_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31) - 256) return SPO_ERR_BAD_SHAPE;
  if (dtype == SPO_DTYPE_BF16 && (d % 64) != 0) return SPO_ERR_BAD_SHAPE;
  if (dtype == SPO_DTYPE_F32 && (d > 4096 || (d % 4) != 0)) return SPO_ERR_BAD_SHAPE;
  return SPO_OK;
}

int32_t spo_loss_fwd(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                     const uint8_t* mask, const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t d,
                     int32_t V, int32_t S, float* loss, float* logp, float* lse, float* coef, float* seq_sums,
                     float* entropy, void* ws, size_t ws_bytes, const spo_params* params, int32_t* d_status,
                     void* stream) {
  int32_t rc = check_loss_shape(dtype, T, d, V);
  if (rc != SPO_OK) return rc;
  if (!params_ok(params) || !W || !loss || !ws || !cu_seqlens || S < 0) return SPO_ERR_INVALID_ARG;
  if (T > 0 && (!H || !y || !logp_old || !a_norm || !logp || !lse || !coef || S < 1)) return SPO_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(W) || !aligned16(y) || !aligned16(logp_old) || !aligned16(cu_seqlens) ||
      !aligned16(a_norm) || !aligned16(logp) || !aligned16(lse) || !aligned16(coef) || !aligned16(entropy) ||
      !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const FwdWs L = fwd_ws_layout(T, d, V, dtype, S);
  if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = forward_launches(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, loss, logp, lse, coef,
                                   seq_sums, entropy, (char*)ws, L, params, d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_loss_bwd(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* lse,
                     const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V, void* dH,
                     int32_t dH_dtype, float* dW, int32_t dW_accumulate, void* ws, size_t ws_bytes,
                     const spo_params* params, int32_t* d_status, void* stream) {
  int32_t rc = check_loss_shape(dtype, T, d, V);
  if (rc != SPO_OK) return rc;
  if (dH_dtype != SPO_DTYPE_F32 && dH_dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (!params_ok(params) || !W || !dW) return SPO_ERR_INVALID_ARG;
  if (T > 0 && (!H || !y || !lse || !coef || !dH)) return SPO_ERR_INVALID_ARG;
  if (dtype == SPO_DTYPE_BF16 && !ws) return SPO_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(W) || !aligned16(y) || !aligned16(lse) || !aligned16(coef) || !aligned16(dH) ||
      !aligned16(dW) || !aligned16(ws))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (dtype == SPO_DTYPE_BF16) {
    const BwdWs L = bwd_ws_layout(T, d, V);
    if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
    e = launch_bwd_bf16(H, W, y, lse, coef, grad_loss, T, d, V, dH, dH_dtype, dW, dW_accumulate, (char*)ws, L,
                        d_status, st);
  } else {
    e = launch_bwd_f32((const float*)H, (const float*)W, y, lse, coef, grad_loss, T, d, V, dH, dH_dtype, dW,
                       dW_accumulate, st);
  }
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

}  // extern "C"

// Behind every slab of dW rows an event, when the caller asked for them (see spo_loss_fwd_bwd_slabs).
// Paths that do not cut the last contraction record all of them at the end.
static cudaError_t record_all(void* const* events, int n, cudaStream_t st) {
  for (int k = 0; k < n; ++k) {
    cudaError_t e = cudaEventRecord((cudaEvent_t)events[k], st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

static int32_t loss_fwd_bwd_impl(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                                 const uint8_t* mask, const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t d,
                                 int32_t V, int32_t S, float grad_loss, float* loss, float* logp, float* lse, float* coef,
                                 float* seq_sums, float* entropy, void* dH, int32_t dH_dtype, float* dW,
                                 int32_t dW_accumulate, void* ws, size_t ws_bytes, const spo_params* params,
                                 int32_t* d_status, void* stream, int32_t n_slabs, void* const* events,
                                 const spo_dw_shards* shards = nullptr) {
  int32_t rc = check_loss_shape(dtype, T, d, V);
  if (shards) {
    if (shards->n_shards < 1 || shards->n_shards > SPO_MAX_DW_SHARDS || shards->rows_per_shard < 1 ||
        (int64_t)shards->n_shards * shards->rows_per_shard < V)
      return SPO_ERR_INVALID_ARG;
    for (int k = 0; k < shards->n_shards; ++k) {
      if (!shards->shard[k]) return SPO_ERR_INVALID_ARG;
      if (!aligned16(shards->shard[k])) return SPO_ERR_BAD_ALIGNMENT;
    }
  }
  if (rc != SPO_OK) return rc;
  if (dH_dtype != SPO_DTYPE_F32 && dH_dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (!params_ok(params) || !W || !loss || !dW || !ws || !cu_seqlens || S < 0) return SPO_ERR_INVALID_ARG;
  if (T > 0 && (!H || !y || !logp_old || !a_norm || !logp || !lse || !coef || !dH || S < 1)) return SPO_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(W) || !aligned16(y) || !aligned16(logp_old) || !aligned16(cu_seqlens) ||
      !aligned16(a_norm) || !aligned16(logp) || !aligned16(lse) || !aligned16(coef) || !aligned16(dH) ||
      !aligned16(dW) || !aligned16(ws) || !aligned16(entropy))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = (cudaStream_t)stream;
  char* w8 = (char*)ws;
  cudaError_t e;
  int slabs_used = 0;                      // slabs the caller's n_slabs comes to (its events 0 .. slabs_used-1 exist)
  if (n_slabs > 0) {
    int64_t bounds[SPO_MAX_DW_SLABS + 1];
    slabs_used = dw_slab_rows(V, d, n_slabs, bounds);
  }
  if (dtype == SPO_DTYPE_BF16 && params->surrogate == SPO_SUR_GSPO) {
    // A response's ratio needs the log-probs of all its tokens, and those may lie in later chunks than
    // the rows whose gradient is being formed: the forward runs to the end first, then the chunked
    // backward (four contractions per token, as spo_loss_fwd followed by spo_loss_bwd).
    const FwdWs Lf = fwd_ws_layout(T, d, V, dtype, S);
    const BwdWs Lb = bwd_ws_layout(T, d, V);
    const size_t off_b = align_up(Lf.total, 256);
    if (ws_bytes < off_b + Lb.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
    if ((e = forward_launches(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, loss, logp, lse, coef,
                              seq_sums, entropy, w8, Lf, params, d_status, st)) != cudaSuccess)
      return cuda_fail(e);
    e = launch_bwd_bf16(H, W, y, lse, coef, grad_loss, T, d, V, dH, dH_dtype, dW, dW_accumulate, w8 + off_b, Lb,
                        d_status, st);
    if (e == cudaSuccess && shards) e = launch_dw_scatter_add(dW, V, d, *shards, st);
    if (e == cudaSuccess && n_slabs > 0) e = record_all(events, slabs_used, st);
    return e == cudaSuccess ? SPO_OK : cuda_fail(e);
  }
  if (dtype == SPO_DTYPE_BF16) {
    const FusedWs L = fused_ws_layout(T, d, V, S);
    if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
    FusedArgs a{};
    a.H = H; a.W = W; a.y = y; a.logp_old = logp_old; a.mask = mask; a.cu_seqlens = cu_seqlens; a.a_norm = a_norm;
    a.T = T; a.d = d; a.V = V; a.S = S; a.grad_loss = grad_loss;
    a.loss = loss; a.logp = logp; a.lse = lse; a.coef = coef; a.seq_sums = seq_sums; a.entropy = entropy;
    a.dH = dH; a.dH_dtype = dH_dtype; a.dW = dW; a.accumulate = dW_accumulate;
    a.params = params; a.d_status = d_status;
    a.n_slabs = n_slabs; a.events = reinterpret_cast<cudaEvent_t*>(const_cast<void**>(events));
    a.shards = shards;
    e = launch_fused_bf16(a, w8, L, st);
    return e == cudaSuccess ? SPO_OK : cuda_fail(e);
  }
  // fp32 inputs: nothing to share between the two halves of the SIMT path; run them back to back
  const FwdWs L = fwd_ws_layout(T, d, V, dtype, S);
  if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  if ((e = forward_launches(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, loss, logp, lse, coef,
                            seq_sums, entropy, w8, L, params, d_status, st)) != cudaSuccess)
    return cuda_fail(e);
  e = launch_bwd_f32((const float*)H, (const float*)W, y, lse, coef, grad_loss, T, d, V, dH, dH_dtype, dW,
                     dW_accumulate, st);
  if (e == cudaSuccess && shards) e = launch_dw_scatter_add(dW, V, d, *shards, st);
  if (e == cudaSuccess && n_slabs > 0) e = record_all(events, slabs_used, st);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

extern "C" {

int32_t spo_loss_fwd_bwd(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                         const uint8_t* mask, const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t d,
                         int32_t V, int32_t S, float grad_loss, float* loss, float* logp, float* lse, float* coef,
                         float* seq_sums, float* entropy, void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                         void* ws, size_t ws_bytes, const spo_params* params, int32_t* d_status, void* stream) {
  return loss_fwd_bwd_impl(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, grad_loss, loss, logp, lse,
                           coef, seq_sums, entropy, dH, dH_dtype, dW, dW_accumulate, ws, ws_bytes, params, d_status,
                           stream, 0, nullptr);
}

int32_t spo_loss_fwd_bwd_scatter(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                                 const uint8_t* mask, const int32_t* cu_seqlens, const float* a_norm, int64_t T,
                                 int32_t d, int32_t V, int32_t S, float grad_loss, float* loss, float* logp, float* lse,
                                 float* coef, float* seq_sums, float* entropy, void* dH, int32_t dH_dtype, float* dW,
                                 int32_t dW_accumulate, void* ws, size_t ws_bytes, const spo_params* params,
                                 int32_t* d_status, void* stream, const spo_dw_shards* shards) {
  if (!shards) return SPO_ERR_INVALID_ARG;
  return loss_fwd_bwd_impl(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, grad_loss, loss, logp, lse,
                           coef, seq_sums, entropy, dH, dH_dtype, dW, dW_accumulate, ws, ws_bytes, params, d_status,
                           stream, 0, nullptr, shards);
}

int32_t spo_dw_slab_rows(int32_t V, int32_t d, int32_t n_wanted, int64_t* row_begin) {
  if (V < 1 || d < 1 || n_wanted < 1 || n_wanted > SPO_MAX_DW_SLABS || !row_begin) return SPO_ERR_INVALID_ARG;
  return dw_slab_rows(V, d, n_wanted, row_begin);
}

int32_t spo_loss_fwd_bwd_slabs(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                               const uint8_t* mask, const int32_t* cu_seqlens, const float* a_norm, int64_t T,
                               int32_t d, int32_t V, int32_t S, float grad_loss, float* loss, float* logp, float* lse,
                               float* coef, float* seq_sums, float* entropy, void* dH, int32_t dH_dtype, float* dW,
                               int32_t dW_accumulate, void* ws, size_t ws_bytes, const spo_params* params,
                               int32_t* d_status, void* stream, int32_t n_wanted, void* const* events) {
  if (n_wanted < 1 || n_wanted > SPO_MAX_DW_SLABS || !events || V < 1 || d < 1) return SPO_ERR_INVALID_ARG;
  int64_t bounds[SPO_MAX_DW_SLABS + 1];
  const int n = dw_slab_rows(V, d, n_wanted, bounds);
  for (int k = 0; k < n; ++k)
    if (!events[k]) return SPO_ERR_INVALID_ARG;
  // dw_slab_rows(n) and the launch must agree on the cut: the launch is asked for the same n_wanted
  return loss_fwd_bwd_impl(H, W, dtype, y, logp_old, mask, cu_seqlens, a_norm, T, d, V, S, grad_loss, loss, logp, lse,
                           coef, seq_sums, entropy, dH, dH_dtype, dW, dW_accumulate, ws, ws_bytes, params, d_status,
                           stream, n_wanted, events);
}

namespace {
struct BwdRowsWs {
  size_t bwd, h_act, dh_act, y_act, lse_act, coef_act, total;
  BwdWs inner;
};
BwdRowsWs bwd_rows_ws_layout(int64_t T_act, int32_t d, int32_t V, int32_t dh_elem) {
  BwdRowsWs L{};
  const int64_t n = T_act > 0 ? T_act : 1;
  L.inner = bwd_ws_layout(T_act, d, V);
  size_t off = 0;
  L.bwd = off;      off = align_up(off + L.inner.total, 256);
  L.h_act = off;    off = align_up(off + (size_t)n * d * 2, 256);
  L.dh_act = off;   off = align_up(off + (size_t)n * d * dh_elem, 256);
  L.y_act = off;    off = align_up(off + (size_t)n * 4, 256);
  L.lse_act = off;  off = align_up(off + (size_t)n * 4, 256);
  L.coef_act = off; off = align_up(off + (size_t)n * 4, 256);
  L.total = off;
  return L;
}
}  // namespace

int32_t spo_loss_active_rows(const float* coef, int64_t T, int32_t* rows, int32_t* d_count, void* ws, size_t ws_bytes,
                             void* stream) {
  if (T < 0 || !d_count || (T > 0 && (!coef || !rows || !ws))) return SPO_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31) - 256) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(coef) || !aligned16(rows) || !aligned16(ws)) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = (cudaStream_t)stream;
  if (T == 0) {
    cudaError_t e0 = cudaMemsetAsync(d_count, 0, sizeof(int32_t), st);
    return e0 == cudaSuccess ? SPO_OK : cuda_fail(e0);
  }
  if (ws_bytes < active_rows_ws_bytes(T)) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = launch_active_rows(coef, nullptr, T, rows, d_count, (int32_t*)ws, st);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

int32_t spo_loss_bwd_rows(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* lse,
                          const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V, const int32_t* rows,
                          int64_t T_act, void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate, void* ws,
                          size_t ws_bytes, const spo_params* params, int32_t* d_status, void* stream) {
  int32_t rc = check_loss_shape(dtype, T, d, V);
  if (rc != SPO_OK) return rc;
  if (dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (dH_dtype != SPO_DTYPE_F32 && dH_dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (!params_ok(params) || !W || !dW || !ws || T_act < 0 || T_act > T) return SPO_ERR_INVALID_ARG;
  if (T > 0 && (!H || !y || !lse || !coef || !dH)) return SPO_ERR_INVALID_ARG;
  if (T_act > 0 && !rows) return SPO_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(W) || !aligned16(y) || !aligned16(lse) || !aligned16(coef) || !aligned16(dH) ||
      !aligned16(dW) || !aligned16(ws) || !aligned16(rows))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const int32_t dh_elem = dH_dtype == SPO_DTYPE_BF16 ? 2 : 4;
  const BwdRowsWs L = bwd_rows_ws_layout(T_act, d, V, dh_elem);
  if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char* w8 = (char*)ws;
  cudaError_t e;
  // rows without gradient get zeros; the others are overwritten by the scatter below
  if (T > 0 && (e = cudaMemsetAsync(dH, 0, (size_t)T * d * dh_elem, st)) != cudaSuccess) return cuda_fail(e);
  void* h_act = w8 + L.h_act;
  void* dh_act = w8 + L.dh_act;
  int32_t* y_act = reinterpret_cast<int32_t*>(w8 + L.y_act);
  float* lse_act = reinterpret_cast<float*>(w8 + L.lse_act);
  float* coef_act = reinterpret_cast<float*>(w8 + L.coef_act);
  if ((e = launch_gather_rows(H, y, lse, coef, rows, T_act, T, d * 2, h_act, y_act, lse_act, coef_act, d_status, st)) != cudaSuccess)
    return cuda_fail(e);
  if ((e = launch_bwd_bf16(h_act, W, y_act, lse_act, coef_act, grad_loss, T_act, d, V, dh_act, dH_dtype, dW,
                           dW_accumulate, w8 + L.bwd, L.inner, d_status, st)) != cudaSuccess)
    return cuda_fail(e);
  if ((e = launch_scatter_rows(dh_act, rows, T_act, T, d * dh_elem, dH, st)) != cudaSuccess) return cuda_fail(e);
  return SPO_OK;
}

int32_t spo_loss_mask_rows(const uint8_t* mask, int64_t T, int32_t* rows, int32_t* d_count, void* ws, size_t ws_bytes,
                           void* stream) {
  if (T < 0 || !d_count || (T > 0 && (!mask || !rows || !ws))) return SPO_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31) - 256) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(mask) || !aligned16(rows) || !aligned16(ws)) return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = (cudaStream_t)stream;
  if (T == 0) {
    cudaError_t e0 = cudaMemsetAsync(d_count, 0, sizeof(int32_t), st);
    return e0 == cudaSuccess ? SPO_OK : cuda_fail(e0);
  }
  if (ws_bytes < active_rows_ws_bytes(T)) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = launch_active_rows(nullptr, mask, T, rows, d_count, (int32_t*)ws, st);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

namespace {
struct FusedRowsWs {
  size_t fused, h_act, dh_act, y_act, lo_act, logp_act, lse_act, coef_act, cu_act, total;
  FusedWs inner;
};
FusedRowsWs fused_rows_ws_layout(int64_t T_act, int32_t d, int32_t V, int32_t S, int32_t dh_elem) {
  FusedRowsWs L{};
  const int64_t n = T_act > 0 ? T_act : 1;
  L.inner = fused_ws_layout(T_act, d, V, S);
  size_t off = 0;
  L.fused = off;    off = align_up(off + L.inner.total, 256);
  L.h_act = off;    off = align_up(off + (size_t)n * d * 2, 256);
  L.dh_act = off;   off = align_up(off + (size_t)n * d * dh_elem, 256);
  L.y_act = off;    off = align_up(off + (size_t)n * 4, 256);
  L.lo_act = off;   off = align_up(off + (size_t)n * 4, 256);
  L.logp_act = off; off = align_up(off + (size_t)n * 4, 256);
  L.lse_act = off;  off = align_up(off + (size_t)n * 4, 256);
  L.coef_act = off; off = align_up(off + (size_t)n * 4, 256);
  L.cu_act = off;   off = align_up(off + (size_t)(S > 0 ? S + 1 : 2) * 4, 256);
  L.total = off;
  return L;
}
}  // namespace

int32_t spo_loss_fwd_bwd_rows(const void* H, const void* W, int32_t dtype, const int32_t* y, const float* logp_old,
                              const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t d, int32_t V,
                              int32_t S, const int32_t* rows, int64_t T_act, float grad_loss, float* loss, float* logp,
                              float* lse, float* coef, float* seq_sums, void* dH, int32_t dH_dtype, float* dW,
                              int32_t dW_accumulate, void* ws, size_t ws_bytes, const spo_params* params,
                              int32_t* d_status, void* stream) {
  int32_t rc = check_loss_shape(dtype, T, d, V);
  if (rc != SPO_OK) return rc;
  if (dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (dH_dtype != SPO_DTYPE_F32 && dH_dtype != SPO_DTYPE_BF16) return SPO_ERR_UNSUPPORTED_DTYPE;
  if (!params_ok(params) || !W || !loss || !dW || !ws || !cu_seqlens || S < 0 || T_act < 0 || T_act > T)
    return SPO_ERR_INVALID_ARG;
  if (params->surrogate == SPO_SUR_GSPO) return SPO_ERR_INVALID_ARG;       // needs whole responses: two-call path
  if (T > 0 && (!H || !y || !logp_old || !a_norm || !logp || !lse || !coef || !dH || S < 1)) return SPO_ERR_INVALID_ARG;
  if (T_act > 0 && !rows) return SPO_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(W) || !aligned16(y) || !aligned16(logp_old) || !aligned16(cu_seqlens) ||
      !aligned16(a_norm) || !aligned16(logp) || !aligned16(lse) || !aligned16(coef) || !aligned16(dH) ||
      !aligned16(dW) || !aligned16(ws) || !aligned16(rows))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  const int32_t dh_elem = dH_dtype == SPO_DTYPE_BF16 ? 2 : 4;
  const FusedRowsWs L = fused_rows_ws_layout(T_act, d, V, S, dh_elem);
  if (ws_bytes < L.total) return SPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  char* w8 = (char*)ws;
  cudaError_t e;
  // rows that are not listed get zeros; the listed ones are overwritten by the scatters below
  if (T > 0) {
    if ((e = cudaMemsetAsync(dH, 0, (size_t)T * d * dh_elem, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemsetAsync(logp, 0, (size_t)T * 4, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemsetAsync(lse, 0, (size_t)T * 4, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemsetAsync(coef, 0, (size_t)T * 4, st)) != cudaSuccess) return cuda_fail(e);
  }
  void* h_act = w8 + L.h_act;
  void* dh_act = w8 + L.dh_act;
  int32_t* y_act = reinterpret_cast<int32_t*>(w8 + L.y_act);
  float* lo_act = reinterpret_cast<float*>(w8 + L.lo_act);
  float* logp_act = reinterpret_cast<float*>(w8 + L.logp_act);
  float* lse_act = reinterpret_cast<float*>(w8 + L.lse_act);
  float* coef_act = reinterpret_cast<float*>(w8 + L.coef_act);
  int32_t* cu_act = reinterpret_cast<int32_t*>(w8 + L.cu_act);
  // the compacted batch: listed rows of H, y, logp_old, and the sequence boundaries among them
  if ((e = launch_gather_rows(H, y, logp_old, logp_old, rows, T_act, T, d * 2, h_act, y_act, lo_act, logp_act, d_status, st)) !=
      cudaSuccess)
    return cuda_fail(e);
  if ((e = launch_compact_cu_seqlens(rows, T_act, cu_seqlens, S, cu_act, st)) != cudaSuccess) return cuda_fail(e);
  FusedArgs a{};
  a.H = h_act; a.W = W; a.y = y_act; a.logp_old = lo_act; a.mask = nullptr; a.cu_seqlens = cu_act; a.a_norm = a_norm;
  a.T = T_act; a.d = d; a.V = V; a.S = S; a.grad_loss = grad_loss;
  a.loss = loss; a.logp = logp_act; a.lse = lse_act; a.coef = coef_act; a.seq_sums = seq_sums; a.entropy = nullptr;
  a.dH = dh_act; a.dH_dtype = dH_dtype; a.dW = dW; a.accumulate = dW_accumulate;
  a.params = params; a.d_status = d_status;
  if ((e = launch_fused_bf16(a, w8 + L.fused, L.inner, st)) != cudaSuccess) return cuda_fail(e);
  if ((e = launch_scatter_scalars(logp_act, lse_act, coef_act, rows, T_act, T, logp, lse, coef, st)) != cudaSuccess)
    return cuda_fail(e);
  if ((e = launch_scatter_rows(dh_act, rows, T_act, T, d * dh_elem, dH, st)) != cudaSuccess) return cuda_fail(e);
  return SPO_OK;
}

int32_t spo_loss_stats(const float* logp, const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                       const float* a_norm, int64_t T, int32_t S, float* out, const spo_params* params, void* stream) {
  if (!params_ok(params) || !out || T < 0 || S < 0) return SPO_ERR_INVALID_ARG;
  if (T > 0 && (!logp || !logp_old || !cu_seqlens || !a_norm || S < 1)) return SPO_ERR_INVALID_ARG;
  if (T >= ((int64_t)1 << 31) - 256) return SPO_ERR_BAD_SHAPE;
  if (!aligned16(logp) || !aligned16(logp_old) || !aligned16(cu_seqlens) || !aligned16(a_norm) || !aligned16(out))
    return SPO_ERR_BAD_ALIGNMENT;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaError_t e = launch_loss_stats(logp, logp_old, mask, cu_seqlens, a_norm, T, S, *params, out,
                                    (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

size_t spo_workspace_bytes(int32_t which, int64_t T, int32_t d, int32_t V, int64_t N, int32_t B, int32_t M) {
  switch (which) {
    case SPO_WS_SAMPLE:
      if (N < 1 || M < 1) return 0;
      return sample_ws_layout(N, M).total;
    case SPO_WS_ADVANTAGES:
      if (B <= kAdvSingleBlockMax) return 256;
      return adv_partial_bytes(B);
    case SPO_WS_UPDATE_REPEATS:
      if (B < 0 || B > kRepeatsMaxBatch) return 0;
      return repeats_ws_layout(B).total;
    case SPO_WS_LOSS_FWD:
      if (T < 0 || V < 1) return 0;
      return fwd_ws_layout(T, d, V, (d % 64) == 0 ? SPO_DTYPE_BF16 : SPO_DTYPE_F32, B).total;
    case SPO_WS_ACTIVE_ROWS:
      if (T < 0) return 0;
      return active_rows_ws_bytes(T);
    case SPO_WS_LOSS_BWD_ROWS:          /* T = number of active rows; sized for an fp32 dH */
      if (T < 0 || V < 1 || d < 1) return 0;
      return bwd_rows_ws_layout(T, d, V, 4).total;
    case SPO_WS_LOSS_BWD:
      if (T < 0 || V < 1 || d < 1) return 0;
      return bwd_ws_layout(T, d, V).total;
    case SPO_WS_LOSS_FWD_BWD_ROWS:      /* T = number of listed rows, B = responses; sized for an fp32 dH */
      if (T < 0 || V < 1 || d < 1 || (d % 64) != 0) return 0;
      return fused_rows_ws_layout(T, d, V, B, 4).total;
    case SPO_WS_LOSS_FWD_BWD: {         /* enough for either element type */
      if (T < 0 || V < 1 || d < 1) return 0;
      const size_t f32 = fwd_ws_layout(T, d, V, SPO_DTYPE_F32, B).total;
      if ((d % 64) != 0) return f32;
      size_t bf16 = fused_ws_layout(T, d, V, B).total;
      const size_t two_call = align_up(fwd_ws_layout(T, d, V, SPO_DTYPE_BF16, B).total, 256) + bwd_ws_layout(T, d, V).total;
      if (two_call > bf16) bf16 = two_call;         // the sequence-level objective runs forward, then backward
      return bf16 > f32 ? bf16 : f32;
    }
    default:
      return 0;
  }
}

int32_t spo_selftest_bounded_wait(uint32_t limit_us, int32_t* reached_end, int32_t* d_status, void* stream) {
  if (!d_status || limit_us == 0 || limit_us > 1000000u) return SPO_ERR_INVALID_ARG;
  if (!device_is_sm100()) return SPO_ERR_UNSUPPORTED_ARCH;
  cudaError_t e = launch_bounded_wait_probe(d_status, limit_us, reached_end, (cudaStream_t)stream);
  return e == cudaSuccess ? SPO_OK : cuda_fail(e);
}

const char* spo_status_string(int32_t status) {
  switch (status) {
    case SPO_OK: return "ok";
    case SPO_ERR_INVALID_ARG: return "invalid argument";
    case SPO_ERR_BAD_SHAPE: return "unsupported shape";
    case SPO_ERR_BAD_ALIGNMENT: return "pointer not 16-byte aligned";
    case SPO_ERR_UNSUPPORTED_DTYPE: return "unsupported element type";
    case SPO_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case SPO_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SPO_ERR_CUDA: return "CUDA error (see spo_last_cuda_error)";
    default: return "unknown status";
  }
}

int32_t spo_last_cuda_error(void) { return g_last_cuda_error; }

int32_t spo_version(void) { return 100; }

}  // extern "C"
