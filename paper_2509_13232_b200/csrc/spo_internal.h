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
int32_t record_cuda_error(cudaError_t e);   // remembers e for spo_last_cuda_error(); returns SPO_ERR_CUDA
int device_is_sm100();                // 1 when the current device is compute capability 10.x

// ---- sampler ------------------------------------------------------------
constexpr int kSampleTile = 2048;     // table entries per partial-sum tile
constexpr int kSuperTile = 1024;      // tiles per second-level sum
// Tables of up to kSmallTableMax prompts take a second form of the same computation, made for latency
// instead of bandwidth: tiles of kSmallTile entries, whose sums every block of the search scans into
// shared memory (the draw needs two dependent global reads instead of some twenty).
constexpr int kSmallTile = 256;
constexpr int kSmallTilesMax = 4096;
constexpr int64_t kSmallTableMax = (int64_t)kSmallTile * kSmallTilesMax;

struct SampleWs {
  size_t super_sums, keys, vals, zeroed_bytes, tile_sums, cand, slot_of, first_draw, total;
  int64_t n_tiles;
  int n_super;
  int64_t hash_slots;
  int small;            // 1: the small-table form (tiles of kSmallTile entries, no second-level sums)
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
// Divergences for the fused advantage + update pass: [B] per batch entry, or [N] per prompt.
struct AdvUpdate { const float* kl; int kl_is_table; };
size_t adv_partial_bytes(int32_t B);   // block records of the two-pass path
cudaError_t launch_advantages(float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                              float* a_raw, float* a_norm, float* stats, void* partials, const spo_params& pr,
                              const AdvUpdate* upd, bool force_two_pass, int32_t* d_status, cudaStream_t st);
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
// (exponent m2 the sums are relative to, in log2 units: the running max of z*log2(e), or on the
// one-pass path the row's fixed reference exponent; sum of 2^(z*log2(e) - m2); target logit or -inf;
// and in `pad` the sum of e*z when the entropy was asked for).
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

// Extra work of the finalisation in the one-pass forward+backward (G == nullptr: none).  With the
// chunk's exponentials e = 2^(z log2e - ref_t) in G and l_t = sum_v e, the logit gradient is
// g[t,v] = rowscale_t (e[t,v] - l_t 1[v = y_t]), rowscale_t = -grad_loss coef_t / l_t: the kernel
// writes rowscale_t and replaces the one entry G[t][y_t] by e - l_t.
struct OnePassFix {
  uint16_t* G;          // bf16 [chunk rows][ldg]
  int64_t ldg;
  int64_t g_row0;       // token row held by row 0 of G
  float* rowscale;      // [T], indexed by token row
  float grad_loss;
};

// need_seq_counts: per-response unmasked counts and the number of responses that have any
cudaError_t launch_fwd_prepare(const uint8_t* mask, int64_t T, const int32_t* cu_seqlens, int32_t S,
                               int need_seq_counts, int32_t* seq_cnt, int32_t* counters, cudaStream_t st);
// Sequence-level objective: coef and loss from the finished logp of all tokens.
cudaError_t launch_seq_level_objective(const float* logp, const float* logp_old, const uint8_t* mask,
                                       const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t S,
                                       const spo_params& pr, const int32_t* counters,
                                       float* seq_coef, double* seq_term, float* coef, float* loss, cudaStream_t st);
cudaError_t launch_fwd_finalize(const FwdPartial* partials, int nsplit, const int32_t* y,
                                const float* logp_old, const uint8_t* mask, const int32_t* cu_seqlens,
                                const float* a_norm, int64_t T, int32_t V, int32_t S,
                                float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                                double* block_sums, int32_t* counters, const int32_t* seq_cnt, const spo_params& pr,
                                int64_t fin_blocks, int32_t* d_status, cudaStream_t st,
                                const FinalizeRange* range = nullptr, const OnePassFix* fix = nullptr);
// out[i][:] = rowscale[t0 + i] * H[t0 + i][:] for i < rows (bf16 rows of row_bytes bytes; a zero factor gives zeros)
cudaError_t launch_scale_rows(const void* H, const float* rowscale, int64_t t0, int64_t rows, int32_t row_bytes,
                              void* out, cudaStream_t st);

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
  size_t g;             // slots x bf16 [chunk_rows][ldg], contiguous: the stored exponentials of one chunk each
  size_t hs;            // slots x bf16 [chunk_rows][d], contiguous: the chunks' rows of H times their row scale
  size_t pre;           // FwdPartial [2][T]: statistics of every row's first vocabulary tile
  size_t rowscale;      // float [T]
  size_t partials;      // FwdPartial [2*nsplit][rows of the chunk]
  size_t progress, block_sums, counters, seq_cnt;
  size_t total;
  int64_t chunk_rows, ldg;
  int64_t fin_blocks;
  int slots;            // chunks whose dW contribution is contracted in one launch (K = their rows together)
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
  // Data-parallel ranks reduce dW while its last contraction still runs: that launch is cut into
  // `n_slabs` slabs of vocabulary rows and events[k] is recorded on the stream behind slab k
  // (0 / NULL: one launch, no events).
  int n_slabs;
  cudaEvent_t* events;
  // Reduce-scatter form (shards != NULL): the last dW contraction adds the finished dW, tile by tile, into
  // the shards that own its vocabulary rows (spo_loss_fwd_bwd_scatter); dW itself is then scratch.
  const spo_dw_shards* shards;
};
// dW[V][d] added into the shards that own its rows (the paths that do not fuse this into a contraction)
cudaError_t launch_dw_scatter_add(const float* dW, int32_t V, int32_t d, const spo_dw_shards& sh, cudaStream_t st);
// Vocabulary-row bounds of the slabs the last dW contraction is cut into: row_begin[0..n] with
// row_begin[0] = 0 and row_begin[n] = V; returns n <= n_wanted (slabs hold whole rounds of row tiles).
int dw_slab_rows(int32_t V, int32_t d, int n_wanted, int64_t* row_begin);
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
                              const float* a_norm, int64_t T, int32_t S, const spo_params& pr, float* out,
                              cudaStream_t st);
cudaError_t launch_compact_cu_seqlens(const int32_t* rows, int64_t n_act, const int32_t* cu_seqlens, int32_t S,
                                      int32_t* cu_act, cudaStream_t st);
cudaError_t launch_scatter_scalars(const float* logp_act, const float* lse_act, const float* coef_act,
                                   const int32_t* rows, int64_t n_act, int64_t T, float* logp, float* lse, float* coef,
                                   cudaStream_t st);
size_t active_rows_ws_bytes(int64_t T);
cudaError_t launch_gather_rows(const void* H, const int32_t* y, const float* lse, const float* coef,
                               const int32_t* rows, int64_t n_act, int64_t T, int32_t row_bytes, void* H_act,
                               int32_t* y_act, float* lse_act, float* coef_act, int32_t* d_status, cudaStream_t st);
cudaError_t launch_scatter_rows(const void* dH_act, const int32_t* rows, int64_t n_act, int64_t T, int32_t row_bytes,
                                void* dH, cudaStream_t st);

cudaError_t launch_bounded_wait_probe(int32_t* d_status, uint32_t limit_us, int32_t* reached_end, cudaStream_t st);

}  // namespace spo
