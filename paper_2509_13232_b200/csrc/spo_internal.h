// Internal declarations shared by the translation units of libspo.
// Nothing here is part of the public ABI (see include/spo.h).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "spo.h"

namespace spo {

// ---- small helpers ------------------------------------------------------
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

int sm_count();                       // SMs of the current device (cached per device)
int device_is_sm100();                // 1 when the current device is compute capability 10.x

// ---- sampler ------------------------------------------------------------
constexpr int kSampleTile = 2048;     // table entries per partial-sum tile
constexpr int kSuperTile = 1024;      // tiles per second-level sum

struct SampleWs {
  size_t super_sums, keys, vals, zeroed_bytes, tile_sums, cand, total;
  int64_t n_tiles;
  int n_super;
  int64_t hash_slots;
};
SampleWs sample_ws_layout(int64_t N, int32_t M);

cudaError_t launch_tracker_init(float* ab, const float* v0, int64_t N, float n0, cudaStream_t st);
cudaError_t launch_sample(const float* ab, int64_t N, const float* u, int32_t M, int32_t B,
                          int32_t* out_ids, float* out_w, char* ws, const SampleWs& L,
                          float eps, int32_t* d_status, cudaStream_t st);

// ---- advantages / tracker ------------------------------------------------
constexpr int kAdvSingleBlockMax = 8192;
int adv_blocks(int32_t B);
cudaError_t launch_advantages_apply(const float* a_raw, int32_t B, float mu, float sigma, float norm_eps, float* a_norm,
                                    cudaStream_t st);
cudaError_t launch_advantages(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                              float* a_raw, float* a_norm, float* stats, char* ws,
                              float norm_eps, int32_t ddof, int32_t* d_status, cudaStream_t st);
cudaError_t launch_tracker_update(float* ab, int64_t N, const int32_t* ids, const float* r,
                                  const float* kl, int kl_is_table, int32_t B,
                                  float rho_min, float rho_max, float d_half,
                                  int32_t* d_status, cudaStream_t st);

constexpr int kRepeatsMaxBatch = 65536;
struct RepeatsWs {
  size_t keys, zeroed_bytes, cur, slot_of, total;
  int64_t hash_slots;
};
RepeatsWs repeats_ws_layout(int32_t B);
cudaError_t launch_tracker_update_repeats(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                                          int kl_is_table, int32_t B, char* ws, const RepeatsWs& L, float rho_min,
                                          float rho_max, float d_half, int32_t* d_status, cudaStream_t st);

// ---- loss: pieces shared by the fp32 and bf16 paths ------------------------
// Forward partial statistics of one vocabulary split, per token row:
// (running max of z*log2(e), sum e of 2^(z*log2(e) - max), target logit or -inf, and in `pad`
// the sum of e*z when the entropy was asked for).
struct FwdPartial { float m2, l, zt; float pad; };

constexpr int kFinalizeThreads = 256;

constexpr size_t kProgressBytes = 1024;   // per-launch progress words of the CTA pairs (bf16 path)

struct FwdWs {
  size_t progress;      // uint32 [256]
  size_t partials;      // FwdPartial [nsplit][T]
  size_t block_sums;    // double [finalize blocks]
  size_t counters;      // int32 [4]: n_tok, ticket, responses with an unmasked token
  size_t seq_cnt;       // int32 [S]: unmasked tokens per response (sequence-mean aggregation)
  size_t seq_coef;      // float [S]: d loss / d logp of a response's unmasked tokens (sequence-level objective)
  size_t seq_term;      // double [S]: objective term of each response (sequence-level objective)
  size_t total;
  int nsplit;
  int64_t fin_blocks;
};
FwdWs fwd_ws_layout(int64_t T, int32_t d, int32_t V, int32_t dtype, int32_t S);

// Rows a finalisation launch covers when the batch is finalised piecewise (one-pass forward+backward).
struct FinalizeRange {
  int64_t t_begin;      // first token row of this launch (a multiple of kFinalizeThreads)
  int64_t part_ld;      // rows between two splits' partials; partial 0 of a split belongs to row t_begin
  int block0;           // index of this launch's first block among all finalisation blocks
  int total_blocks;     // finalisation blocks over the whole batch; the last one to finish folds the loss
  int last;             // 1 when this launch covers the final rows (per-response sums are taken then)
};

// need_seq_counts: per-response unmasked counts and the number of responses that have any
cudaError_t launch_fwd_prepare(const uint8_t* mask, int64_t T, const int32_t* cu_seqlens, int32_t S,
                               int need_seq_counts, int32_t* seq_cnt, int32_t* counters, cudaStream_t st);
// Sequence-level objective: coef and loss from the finished logp of all tokens.
cudaError_t launch_seq_level_objective(const float* logp, const float* logp_old, const uint8_t* mask,
                                       const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t S,
                                       float clip_lo, float clip_hi, const int32_t* counters, int32_t global_responses,
                                       float* seq_coef, double* seq_term, float* coef, float* loss, cudaStream_t st);
cudaError_t launch_fwd_finalize(const FwdPartial* partials, int nsplit, const int32_t* y,
                                const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                                const float* a_norm, int64_t T, int32_t V, int32_t S,
                                float clip_lo, float clip_hi,
                                float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                                double* block_sums, int32_t* counters, const int32_t* seq_cnt, int agg_mode,
                                int surrogate, int32_t global_tokens, int32_t global_responses,
                                int64_t fin_blocks, int32_t* d_status, cudaStream_t st,
                                const FinalizeRange* range = nullptr);

// fp32 SIMT path
cudaError_t launch_fwd_f32(const float* H, const float* W, const int32_t* y, int64_t T, int32_t d, int32_t V,
                           FwdPartial* partials, cudaStream_t st);
cudaError_t launch_bwd_f32(const float* H, const float* W, const int32_t* y, const float* lse,
                           const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V,
                           void* dH, int32_t dH_dtype, float* dW, int accumulate, cudaStream_t st);

// bf16 tensor-core path
struct BwdWs {
  size_t g;             // bf16 [chunk_rows][ldg]
  size_t progress;      // uint32 [256]
  size_t total;
  int64_t chunk_rows;   // token rows per chunk (multiple of 128)
  int64_t ldg;          // row pitch of g in elements (multiple of 256)
};
BwdWs bwd_ws_layout(int64_t T, int32_t d, int32_t V);

// one-pass forward+backward (bf16)
struct FusedWs {
  size_t g;             // n_buf x bf16 [chunk_rows][ldg]: e, then g, of one chunk each
  size_t ref;           // n_buf x float [ldg/64][chunk_rows]: reference exponents of e
  size_t g_bytes, ref_bytes;   // size of one of them
  size_t partials;      // FwdPartial [2*nsplit][rows of the chunk]
  size_t progress, block_sums, counters, seq_cnt;
  size_t total;
  int64_t chunk_rows, ldg;
  int64_t fin_blocks;
  int n_buf;            // 2 when there is more than one chunk (chunks are software-pipelined), else 1
};
FusedWs fused_ws_layout(int64_t T, int32_t d, int32_t V, int32_t S);
struct FusedArgs {
  const void *H, *W;
  const int32_t* y;
  const float* logp_old;
  const uint8_t* mask;
  const int32_t* cu_seqlens;
  const float* a_norm;
  int64_t T;
  int32_t d, V, S;
  float grad_loss;
  float *loss, *logp, *lse, *coef, *seq_sums, *entropy;
  void* dH;
  int32_t dH_dtype;
  float* dW;
  int accumulate;
  const spo_params* params;
  int32_t* d_status;
};
cudaError_t launch_fused_bf16(const FusedArgs& a, char* ws, const FusedWs& L, cudaStream_t st);

cudaError_t launch_fwd_bf16(const void* H, const void* W, const int32_t* y, int64_t T, int32_t d, int32_t V,
                            FwdPartial* partials, int nsplit, int want_entropy, uint32_t* progress, int32_t* d_status,
                            cudaStream_t st);
cudaError_t launch_bwd_bf16(const void* H, const void* W, const int32_t* y, const float* lse,
                            const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V,
                            void* dH, int32_t dH_dtype, float* dW, int accumulate,
                            char* ws, const BwdWs& L, int32_t* d_status, cudaStream_t st);

// row compaction for the backward
// rows listed: coef[t] != 0 (coef given) or mask[t] != 0 (mask given, coef NULL)
cudaError_t launch_active_rows(const float* coef, const uint8_t* mask, int64_t T, int32_t* rows, int32_t* d_count,
                               int32_t* block_cnt, cudaStream_t st);
cudaError_t launch_loss_stats(const float* logp, const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                              const float* a_norm, int64_t T, int32_t S, float clip_lo, float clip_hi, float* out,
                              cudaStream_t st);
cudaError_t launch_compact_cu_seqlens(const int32_t* rows, int64_t n_act, const int32_t* cu_seqlens, int32_t S,
                                      int32_t* cu_act, cudaStream_t st);
cudaError_t launch_scatter_scalars(const float* logp_act, const float* lse_act, const float* coef_act,
                                   const int32_t* rows, int64_t n_act, float* logp, float* lse, float* coef,
                                   cudaStream_t st);
size_t active_rows_ws_bytes(int64_t T);
cudaError_t launch_gather_rows(const void* H, const int32_t* y, const float* lse, const float* coef,
                               const int32_t* rows, int64_t n_act, int32_t row_bytes, void* H_act, int32_t* y_act,
                               float* lse_act, float* coef_act, cudaStream_t st);
cudaError_t launch_scatter_rows(const void* dH_act, const int32_t* rows, int64_t n_act, int32_t row_bytes, void* dH,
                                cudaStream_t st);

cudaError_t launch_bounded_wait_probe(int32_t* d_status, uint32_t limit_us, int32_t* reached_end, cudaStream_t st);

}  // namespace spo
