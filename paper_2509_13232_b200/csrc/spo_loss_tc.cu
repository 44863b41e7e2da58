// bf16 loss forward / backward on the 5th-generation tensor cores (sm_100a).
//
// One persistent, warp-specialised kernel template does every contraction of the path:
//   FWD : S = H W^T tile by tile; epilogue keeps an online (max, sum-exp, target logit)
//         per token row in registers across the vocabulary tiles of its split.
//   G   : the same contraction for one chunk of token rows; epilogue turns each logit
//         into g = c_t (1[v=y_t] - e^{z-lse_t}) and writes it as bf16 into the chunk buffer.
//   E   : the same contraction again, for the one-pass forward+backward: epilogue sums the
//         row's exponentials AND writes every logit of the chunk as e = 2^(z log2e - ref_t),
//         bf16, against one reference exponent per token row that is fixed before the sweep.
//         With l_t = sum_v e the softmax is p = e / l_t, so the logit gradient factors as
//         g[t,v] = rowscale_t * (e[t,v] - l_t 1[v = y_t]): the finalisation kernel patches the
//         one target entry per row, and a per-row scale (in DH's epilogue, and applied to the
//         rows of H that DW reads) does the rest -- the stored chunk is never rewritten and the
//         backward needs no second logits contraction.
//   DH  : dH_chunk = G W        (A = G, K-major;  B = W read as an N-major operand)
//   DW  : dW (+)= G^T H_chunk   (A = G read as an M-major operand; B = H, N-major)
//
// CTAs run as pairs (a cluster of two SMs, tcgen05 cta_group::2).  A pair owns a
// 256 x 512 output tile: per 64-deep k-block each CTA stages 128 rows of A and its
// half (2 x 128 columns) of B, and the leader issues two 256x256x16 MMAs per k-step
// that share the A operand and fill the two 256-column halves of tensor memory.
// The wide tile is what keeps the L2 -> shared-memory traffic (48 KB per 256x256x64
// block of MACs) under the L2 bandwidth; the price is that the accumulator is not
// double-buffered, so the epilogue is kept short: eight warps drain it in parallel.
//
// Pipeline per CTA (one CTA per SM, 352 threads):
//   warp 0 : allocates tensor memory; lane 0 issues the TMA loads (128-byte swizzle)
//            of this CTA's operand parts into its 4-stage shared-memory ring; completion
//            is signalled on the "full" mbarrier of the pair's leader CTA.
//   warp 1 : (leader CTA only) lane 0 issues tcgen05.mma (bf16 -> fp32);
//            tcgen05.commit, multicast to both CTAs, releases the stage ("empty") and,
//            after the last k-block, publishes the accumulator ("tfull").
//   warps 2-9 : epilogue; each owns the 32 accumulator lanes its warp id selects and one
//            256-column half, reads them with tcgen05.ld and applies the mode's fused
//            epilogue, then releases the accumulator ("tempty", on the leader).
//   warp 10 : (leader CTA only) pacer: publishes how many k-blocks the pair has loaded, reads the
//            other pairs' counts and tells warp 0 how far it may run ahead of the slowest, so
//            that pairs sweeping the same operand tiles find them in L2.
// Every mbarrier wait is bounded: when it runs out the CTA raises SPO_DEV_TIMEOUT,
// all roles leave their loops, tensor memory is released and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include <atomic>

#include "spo_internal.h"

namespace spo {

namespace {

constexpr int CG = 2;                   // CTAs per MMA group (cluster size)
constexpr int BM = 128;                 // rows of A (and accumulator lanes) per CTA
constexpr int GROUP_M = BM * CG;        // rows of one output tile
constexpr int HALF_N = 256;             // columns of one MMA / one accumulator half
constexpr int BN = 2 * HALF_N;          // columns of one output tile
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;                 // 16 KB
constexpr int BSUB_ROWS = HALF_N / CG;               // B columns per CTA per half (128)
constexpr int BSUB_BYTES = BSUB_ROWS * BK * 2;       // 16 KB
constexpr int STAGE_BYTES = A_BYTES + 2 * BSUB_BYTES;  // 48 KB
constexpr int EPI_WARPS = 8;
constexpr int PACER_WARP = 2 + EPI_WARPS;              // last warp: keeps the pairs' loads close together in time
constexpr int NUM_THREADS = 32 * (3 + EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr int STAGING_BYTES = 4096;                    // per epilogue warp: 32 rows x 128 bytes, for coalesced stores
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256 + EPI_WARPS * STAGING_BYTES;
constexpr unsigned long long kWaitLimitNs = 4000000000ull;
constexpr int kEpilogueSleepNs = 64;
constexpr int kProducerSleepNs = 32;
// Between two looks at the other pairs' progress.  The 74 counters share three cache lines that every
// pacer reads and writes, i.e. one L2 slice serves them all beside its share of the operand traffic:
// looks every 32 ns cost 4 % of the step and a loop with its loads issued back to back 50 %; 256, 1024 and
// 4096 ns agree within 0.2 %; 16 384 ns (longer than the window lasts) stalls the pairs.
constexpr int kPacerSleepNs = 1024;                     // between two looks at the other pairs' progress
constexpr uint32_t kPacerMaxSpins = 1u << 24;          // the pacer gives up (and lets everyone run free) after this many looks
constexpr int kLagCut = 8;                             // pairs more than this many windows behind are not waited for
constexpr int kHoldTries = 2048;                       // x 64 ns: longest time a producer holds back for the slowest pair

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRefMargin = 40.0f;     // binary orders between a row's reference exponent and its first tile's maximum

enum : int { MODE_FWD = 0, MODE_G = 1, MODE_DH = 2, MODE_DW = 3, MODE_E = 4 };
constexpr int kMaxDwShards = SPO_MAX_DW_SHARDS;

struct GemmParams {
  int m_tiles, n_tiles, nsplit, per_split;   // work decomposition: unit = (row tile, split of the column tiles)
  int k_blocks;                              // K / 64, rounded up
  int a_row0;                                // added to A's row coordinate (K-major A) or k coordinate (M-major A)
  int b_k0;                                  // added to B's k coordinate (N-major B)
  int64_t rows_valid;                        // rows of the output that exist (tokens or vocabulary rows)
  int32_t cols_valid;                        // columns of the output that exist (V or d)
  int64_t out_row0;                          // first output row of tile row 0 (token offset of the chunk)
  // FWD / G
  const int32_t* y;
  const float* lse;
  const float* coef;
  float grad_loss;
  FwdPartial* partials;
  int64_t T;                                 // stride between the splits' partials (rows they cover)
  int64_t part_row0;                         // global row that partial 0 of a split belongs to
  __nv_bfloat16* G;
  int64_t ldg;
  const FwdPartial* pre;                     // E: statistics of every row's first vocabulary tile, [2][pre_ld] (both halves)
  int64_t pre_ld;
  const float* rowscale;                     // DH (one-pass): factor of each output row, indexed like the output; NULL = none
  int m_tile0;                               // added to every unit's row tile (a launch that covers a slab of row tiles)
  // DW, reduce-scatter form: instead of going to `out`, every tile (plus what `out` holds, when accumulating)
  // is ADDED into the shard that owns its vocabulary rows; shard k = rows [k shard_rows, (k+1) shard_rows)
  float* shard[kMaxDwShards];
  int n_shards;                              // 0: plain output
  int64_t shard_rows;
  // DH / DW
  void* out;
  int out_bf16;
  int64_t ldo;
  int accumulate;
  int32_t* d_status;
  // Soft lock-step between CTA pairs: progress[g] = k-blocks whose loads pair g has issued, ~0u when done;
  // a pair holds its loads back while it is more than `window` k-blocks ahead of the slowest pair.
  uint32_t* progress;
  int window;
};

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Arrive on a barrier given by a shared::cluster address (possibly in the peer CTA).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Cluster-scope acquire: the barriers here are arrived on by the peer CTA or by tcgen05.commit.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when the wait ran out or another role already gave up.
// SLEEP_NS > 0 backs off between polls (roles that wait long and need not react within nanoseconds).
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* d_status,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  uint32_t spins = 0;
  unsigned long long t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        if (d_status) atomicOr(d_status, SPO_DEV_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// TMA tile load into this CTA's shared memory; completion bytes are counted on `bar`, a
// shared::cluster address that belongs to the pair's leader CTA.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc)
      : "memory");
}
// Arrive, once all MMAs issued so far have completed, on the barrier at this offset in both CTAs.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
// Wait for outstanding tensor-memory loads.  The destination registers are named as in/out operands
// so that the compiler cannot schedule any use of them ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&v)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                 "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                 "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                 "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  tmem_ld32_nowait(taddr, v);
  tmem_wait_ld(v);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// The lane that owns tile row `lane` deposits its 128 bytes (eight 16-byte pieces) into the warp's
// staging buffer; piece c of row r sits at position c ^ (r & 7) so that both this row-wise write and
// the piece-wise read-back below are free of bank conflicts.
__device__ __forceinline__ void stage_put(uint8_t* stage, int lane, const uint4 (&piece)[8]) {
  __syncwarp();                                   // earlier read-backs of this buffer are done
#pragma unroll
  for (int c = 0; c < 8; ++c)
    *reinterpret_cast<uint4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4)) = piece[c];
  __syncwarp();
}
// Read-back i (0..7): lanes 8j..8j+7 fetch the eight pieces of row 4i + j, so one warp-wide global
// access covers four whole 128-byte rows.
__device__ __forceinline__ uint4 stage_get(const uint8_t* stage, int lane, int i, int& r, int& c) {
  r = 4 * i + (lane >> 3);
  c = lane & 7;
  return *reinterpret_cast<const uint4*>(stage + r * 128 + ((c ^ (r & 7)) << 4));
}

// g = c_t (1[v = y_t] - 2^(z log2e - lse_t log2e)) for 32 consecutive columns, packed to bf16.
__device__ __forceinline__ void g_values(const uint32_t (&v)[32], int col0, float c, float lse2, int yt,
                                         int cols_valid, uint4* out4) {
  float g[32];
  if (c != 0.0f) {
    const float nc = -c;
#pragma unroll
    for (int j = 0; j < 32; ++j) g[j] = nc * fast_exp2(fmaf(__uint_as_float(v[j]), kLog2e, -lse2));
    if (yt >= col0 && yt < col0 + 32) {
      const int jj = yt - col0;
#pragma unroll
      for (int j = 0; j < 32; ++j) if (j == jj) g[j] += c;
    }
    if (col0 + 32 > cols_valid) {
#pragma unroll
      for (int j = 0; j < 32; ++j) if (col0 + j >= cols_valid) g[j] = 0.0f;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) g[j] = 0.0f;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q)
    out4[q] = make_uint4(pack_bf16(g[8 * q + 0], g[8 * q + 1]), pack_bf16(g[8 * q + 2], g[8 * q + 3]),
                         pack_bf16(g[8 * q + 4], g[8 * q + 5]), pack_bf16(g[8 * q + 6], g[8 * q + 7]));
}

// Two floats to a bf16 pair, infinities replaced by the largest finite value (stored exponentials
// of a row whose logits outrun the reference must not become Inf: Inf times a zero row scale is NaN).
__device__ __forceinline__ uint32_t pack_bf16_finite(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.satfinite.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ void bf16_values_finite(const uint32_t (&v)[32], uint4* out4) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    out4[q] = make_uint4(pack_bf16_finite(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])),
                         pack_bf16_finite(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                         pack_bf16_finite(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                         pack_bf16_finite(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
}

__device__ __forceinline__ void bf16_values(const uint32_t (&v)[32], uint4* out4) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    out4[q] = make_uint4(pack_bf16(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])),
                         pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                         pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                         pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
}


// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// lbo / sbo in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate, bf16 A and B, M = 256 over the pair, N = 256.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(HALF_N >> 3) << 17) | ((uint32_t)(GROUP_M >> 4) << 24);
}


struct Unit { int m_tile, n_begin, n_end; };
__device__ __forceinline__ Unit unit_of(int u, const GemmParams& p) {
  Unit r;
  const int split = u % p.nsplit;
  r.m_tile = u / p.nsplit + p.m_tile0;
  r.n_begin = split * p.per_split;
  r.n_end = min(r.n_begin + p.per_split, p.n_tiles);
  return r;
}

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
// ENT (FWD / E): also accumulate sum_v e z per row, from which the finalisation forms the entropy of
// the row's softmax, lse - sum_v p z (one more multiply-add per logit; a separate instantiation so that
// the kernels without it stay as they are).
template <int MODE, bool ENT = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
spo_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  constexpr bool A_MN = (MODE == MODE_DW);
  constexpr bool B_MN = (MODE == MODE_DH || MODE == MODE_DW);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bars = base + STAGES * STAGE_BYTES;
  const uint32_t full0 = bars, empty0 = bars + 8 * STAGES, tfull = bars + 16 * STAGES, tempty = tfull + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + STAGES * STAGE_BYTES + 16 * STAGES + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + STAGES * STAGE_BYTES + 16 * STAGES + 24);
  volatile uint32_t* pace_mine = reinterpret_cast<volatile uint32_t*>(gen + STAGES * STAGE_BYTES + 16 * STAGES + 32);
  volatile uint32_t* pace_limit = pace_mine + 1;   // k-blocks this pair's producer may have issued (pacer -> producer)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                    // 0 = leader of the pair
  const int group = blockIdx.x / CG, n_groups = gridDim.x / CG;
  const int total_units = p.m_tiles * p.nsplit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(tfull, 1);
    mbar_init(tempty, EPI_WARPS * CG);
    *abort_flag = 0;
    *pace_mine = 0;
    *pace_limit = p.progress ? (uint32_t)p.window : 0xFFFFFFFFu;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                       // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // Lane 0 issues the loads.  Before each k-block it tells the pacer warp how far it is and holds
    // back while it is ahead of what the pacer allows (the slowest pair's count plus `window`
    // k-blocks): pairs that sweep the same operand tiles then stay close enough in time for those
    // tiles to be served from L2 instead of being streamed from HBM once per pair (without any pacing
    // the forward at 244k tokens read 0.8 TB from HBM per launch, with it 0.12 TB; dH at one look per
    // tile read 17 GB per chunk, at a window of 32 k-blocks 8 GB).  Both words are in shared memory,
    // so the loop pays two shared-memory accesses per k-block; the looks at the other pairs are the
    // pacer's.  The hold is bounded and advisory (after ~0.13 ms the pair goes on regardless), so
    // it cannot dead-lock, and finished pairs publish ~0u so that they never hold anyone back.
    uint32_t it = 0;
    int ok = 1;
    const bool paced = (rank == 0) && p.progress != nullptr;
    for (int u = group; u < total_units; u += n_groups) {
      const Unit un = unit_of(u, p);
      const int row_base = un.m_tile * GROUP_M + (int)rank * BM;       // this CTA's rows of the tile
      for (int n = un.n_begin; n < un.n_end; ++n) {
        const int col_base = n * BN + (int)rank * BSUB_ROWS;           // this CTA's columns of half 0
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          if (paced && lane == 0 && ok) {
            *pace_mine = it;
            for (int tries = 0; tries < kHoldTries && it > *pace_limit; ++tries) __nanosleep(64);
          }
          if (lane == 0 && ok) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait<kProducerSleepNs>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.d_status)) {
              ok = 0;
            } else {
              const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
              if (rank == 0) mbar_expect_tx(full0 + 8 * s, CG * STAGE_BYTES);   // both CTAs' bytes land on the leader's barrier
              const uint32_t fb = map_to_cta(full0 + 8 * s, 0);
              if (!A_MN) {
                tma_load_2d(sa, &tmA, kb * BK, p.a_row0 + row_base, fb);
              } else {
#pragma unroll
                for (int b = 0; b < BM / 64; ++b)
                  tma_load_2d(sa + b * 8192, &tmA, row_base + b * 64, p.a_row0 + kb * BK, fb);
              }
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const uint32_t sbh = sb + h * BSUB_BYTES;
                const int col = col_base + h * HALF_N;
                if (!B_MN) {
                  tma_load_2d(sbh, &tmB, kb * BK, col, fb);
                } else {
#pragma unroll
                  for (int b = 0; b < BSUB_ROWS / 64; ++b)
                    tma_load_2d(sbh + b * 8192, &tmB, col + b * 64, p.b_k0 + kb * BK, fb);
                }
              }
            }
          }
        }
      }
    }
    __syncwarp();
    if (paced && lane == 0) *pace_mine = 0xFFFFFFFFu;                  // done: the pacer publishes it and stops
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc(A_MN, B_MN);
      uint32_t it = 0, tile = 0;
      bool ok = true;
      for (int u = group; u < total_units && ok; u += n_groups) {
        const Unit un = unit_of(u, p);
        for (int n = un.n_begin; n < un.n_end && ok; ++n, ++tile) {
          if (!mbar_wait(tempty, (tile & 1u) ^ 1u, abort_flag, p.d_status)) { ok = false; break; }
          tc_fence_after();
          for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.d_status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
            for (int j = 0; j < BK / 16; ++j) {
              const uint64_t da = A_MN ? smem_desc(sa + j * 2048, 8192, 1024) : smem_desc(sa + j * 32, 16, 1024);
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const uint32_t sbh = sb + h * BSUB_BYTES;
                const uint64_t db = B_MN ? smem_desc(sbh + j * 2048, 8192, 1024) : smem_desc(sbh + j * 32, 16, 1024);
                umma_bf16(tmem_base + h * HALF_N, da, db, idesc, (kb | j) != 0 ? 1u : 0u);
              }
            }
            umma_commit(empty0 + 8 * s);
          }
          if (ok) umma_commit(tfull);
        }
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int quarter = warp & 3;                            // tensor-memory lanes this warp may read
    const int half = (warp - 2) >> 2;                        // which 256-column half of the tile
    const int row = (int)rank * BM + quarter * 32 + lane;    // row of the pair's tile
    const int warp_row0 = (int)rank * BM + quarter * 32;     // tile row of the warp's first lane
    uint8_t* stage = gen + STAGES * STAGE_BYTES + 256 + (warp - 2) * STAGING_BYTES;
    const uint32_t tempty_leader = map_to_cta(tempty, 0);
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + half * HALF_N;
    uint32_t tile = 0;
    bool ok = true;
    for (int u = group; u < total_units && ok; u += n_groups) {
      const Unit un = unit_of(u, p);
      const int64_t grow = p.out_row0 + (int64_t)un.m_tile * GROUP_M + row;   // global output row of this lane
      const int64_t grow_warp0 = grow - lane;                                  // ... and of the warp's first lane
      const bool row_ok = grow < p.rows_valid;
      // per-row state
      float m2 = -CUDART_INF_F, l = 0.0f, zt = -CUDART_INF_F;             // FWD
      float ez = 0.0f;                                                     // ENT: sum e z relative to m2
      int32_t yt = -1;
      float c = 0.0f, lse2 = 0.0f;                                         // G
      float rs = 1.0f;                                                     // DH: factor of this lane's output row
      if (MODE == MODE_FWD || MODE == MODE_G || MODE == MODE_E) {
        if (row_ok) yt = p.y[grow];
        if (MODE == MODE_G && row_ok) { c = p.grad_loss * p.coef[grow]; lse2 = p.lse[grow] * kLog2e; }
        if (MODE == MODE_E) {
          // Reference exponent of the row: the largest logit of its first vocabulary tile (found by a
          // short launch beforehand) plus a margin, the same for every pair and column half that works
          // on the row.  Exponentials are taken against it without a running maximum: bf16 and fp32
          // keep their relative precision at any magnitude, so all that matters is that nothing
          // overflows (row maximum up to kRefMargin + 109 binary orders above the first tile's) and
          // that entries worth keeping do not underflow (anything within 126 - kRefMargin orders
          // below the first tile's maximum survives).
          m2 = row_ok ? fmaxf(p.pre[grow].m2, p.pre[p.pre_ld + grow].m2) + kRefMargin : 0.0f;
        }
      }
      if (MODE == MODE_DH && p.rowscale && row_ok) rs = p.rowscale[grow];
      for (int n = un.n_begin; n < un.n_end && ok; ++n, ++tile) {
        {                                   // one lane polls (with backoff); the warp reconverges on the outcome
          int good = 1;
          if (lane == 0) good = mbar_wait<kEpilogueSleepNs>(tfull, tile & 1u, abort_flag, p.d_status) ? 1 : 0;
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
        }
        tc_fence_after();
        const int col_half = n * BN + half * HALF_N;
        if (MODE == MODE_FWD) {
#pragma unroll 1
          for (int ch = 0; ch < HALF_N / 32; ++ch) {
            const int col0 = col_half + ch * 32;
            if (col0 >= p.cols_valid) break;                           // nothing valid further right
            uint32_t v[32];
            tmem_ld32(taddr + ch * 32, v);
            if (col0 + 32 > p.cols_valid) {                            // ragged last chunk of the vocabulary
              // (with ENT a large finite value instead of -inf: its e is 0 either way and 0 * z stays 0)
              const float fill = ENT ? -1.0e30f : -CUDART_INF_F;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j >= p.cols_valid) v[j] = __float_as_uint(fill);
            }
            float mx0 = __uint_as_float(v[0]), mx1 = __uint_as_float(v[1]);
#pragma unroll
            for (int j = 2; j < 32; j += 2) {
              mx0 = fmaxf(mx0, __uint_as_float(v[j]));
              mx1 = fmaxf(mx1, __uint_as_float(v[j + 1]));
            }
            const float mn = fmaxf(m2, fmaxf(mx0, mx1) * kLog2e);
            const float neg = -mn;
            float s0 = 0.0f, s1 = 0.0f, t0 = 0.0f, t1 = 0.0f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const float e0 = fast_exp2(fmaf(__uint_as_float(v[j]), kLog2e, neg));
              const float e1 = fast_exp2(fmaf(__uint_as_float(v[j + 1]), kLog2e, neg));
              s0 += e0;
              s1 += e1;
              if (ENT) {
                t0 = fmaf(e0, __uint_as_float(v[j]), t0);
                t1 = fmaf(e1, __uint_as_float(v[j + 1]), t1);
              }
            }
            const float down = fast_exp2(m2 - mn);
            l = fmaf(l, down, s0 + s1);
            if (ENT) ez = fmaf(ez, down, t0 + t1);
            m2 = mn;
            if (yt >= col0 && yt < col0 + 32) {
              const int jj = yt - col0;
#pragma unroll
              for (int j = 0; j < 32; ++j) if (j == jj) zt = __uint_as_float(v[j]);
            }
          }
        } else if (MODE == MODE_E) {
          // Sum of the row's exponentials (and sum e z with ENT) and the stored exponentials in one
          // pass, all against the row's fixed reference m2: no running maximum, no rescaling.
          __nv_bfloat16* obase = p.G + ((int64_t)(un.m_tile - p.m_tile0) * GROUP_M + warp_row0) * p.ldg;
          const float neg = -m2;
#pragma unroll 1
          for (int r2 = 0; r2 < HALF_N / 64; ++r2) {
            const int col0 = col_half + r2 * 64;
            uint4 piece[8];
            if (col0 < p.cols_valid) {
              uint32_t v0[32], v1[32];
              tmem_ld32_nowait(taddr + r2 * 64, v0);
              tmem_ld32_nowait(taddr + r2 * 64 + 32, v1);
              tmem_wait_ld(v0);
              tmem_wait_ld(v1);
              if (col0 + 64 > p.cols_valid) {                          // ragged end of the vocabulary: e = 0
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  // (with ENT a large finite value instead of -inf: its e is 0 either way and 0 * z stays 0)
                  const float fill = ENT ? -1.0e30f : -CUDART_INF_F;
                  if (col0 + j >= p.cols_valid) v0[j] = __float_as_uint(fill);
                  if (col0 + 32 + j >= p.cols_valid) v1[j] = __float_as_uint(fill);
                }
              }
              if (yt >= col0 && yt < col0 + 64) {
                const int jj = yt - col0;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  if (j == jj) zt = __uint_as_float(v0[j]);
                  if (j + 32 == jj) zt = __uint_as_float(v1[j]);
                }
              }
              float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f, t0 = 0.0f, t1 = 0.0f;
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const float e0 = fast_exp2(fmaf(__uint_as_float(v0[j]), kLog2e, neg));
                const float e1 = fast_exp2(fmaf(__uint_as_float(v0[j + 1]), kLog2e, neg));
                const float e2 = fast_exp2(fmaf(__uint_as_float(v1[j]), kLog2e, neg));
                const float e3 = fast_exp2(fmaf(__uint_as_float(v1[j + 1]), kLog2e, neg));
                s0 += e0; s1 += e1; s2 += e2; s3 += e3;
                if (ENT) {
                  t0 = fmaf(e0, __uint_as_float(v0[j]), fmaf(e1, __uint_as_float(v0[j + 1]), t0));
                  t1 = fmaf(e2, __uint_as_float(v1[j]), fmaf(e3, __uint_as_float(v1[j + 1]), t1));
                }
                v0[j] = __float_as_uint(e0); v0[j + 1] = __float_as_uint(e1);
                v1[j] = __float_as_uint(e2); v1[j + 1] = __float_as_uint(e3);
              }
              l += (s0 + s1) + (s2 + s3);
              if (ENT) ez += t0 + t1;
              bf16_values_finite(v0, piece);
              bf16_values_finite(v1, piece + 4);
            } else {                                                   // pad columns: e = 0
#pragma unroll
              for (int q = 0; q < 8; ++q) piece[q] = make_uint4(0u, 0u, 0u, 0u);
            }
            stage_put(stage, lane, piece);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              int r, cc;
              const uint4 val = stage_get(stage, lane, i, r, cc);
              if (grow_warp0 + r < p.rows_valid) {
                // streaming store: the chunk buffer is next read by another launch, and lines that stayed in
                // L2 would push out the row strips of H that every tile of this sweep re-reads
                __stcs(reinterpret_cast<uint4*>(obase + (int64_t)r * p.ldg + col0 + cc * 8), val);
              }
            }
          }
        } else if (MODE == MODE_G || (MODE == MODE_DH && p.out_bf16)) {
          // bf16 outputs: 64 columns (128 bytes per row) per staging round
          __nv_bfloat16* obase = MODE == MODE_G
              ? p.G + ((int64_t)un.m_tile * GROUP_M + warp_row0) * p.ldg
              : reinterpret_cast<__nv_bfloat16*>(p.out) + grow_warp0 * p.ldo;
          const int64_t ld = MODE == MODE_G ? p.ldg : p.ldo;
#pragma unroll 1
          for (int r2 = 0; r2 < HALF_N / 64; ++r2) {
            const int col0 = col_half + r2 * 64;
            if (MODE != MODE_G && col0 >= p.cols_valid) break;
            uint32_t v0[32], v1[32];
            tmem_ld32_nowait(taddr + r2 * 64, v0);
            tmem_ld32_nowait(taddr + r2 * 64 + 32, v1);
            tmem_wait_ld(v0);
            tmem_wait_ld(v1);
            uint4 piece[8];
            if (MODE == MODE_G) {
              g_values(v0, col0, c, lse2, yt, p.cols_valid, piece);
              g_values(v1, col0 + 32, c, lse2, yt, p.cols_valid, piece + 4);
            } else {
              if (p.rowscale) {                    // one-pass path: the row's factor (a zero factor gives exact zeros)
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  v0[j] = __float_as_uint(rs == 0.0f ? 0.0f : __uint_as_float(v0[j]) * rs);
                  v1[j] = __float_as_uint(rs == 0.0f ? 0.0f : __uint_as_float(v1[j]) * rs);
                }
              }
              bf16_values(v0, piece);
              bf16_values(v1, piece + 4);
            }
            stage_put(stage, lane, piece);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              int r, cc;
              const uint4 val = stage_get(stage, lane, i, r, cc);
              if (grow_warp0 + r < p.rows_valid) {
                uint4* dst = reinterpret_cast<uint4*>(obase + (int64_t)r * ld + col0 + cc * 8);
                if (MODE == MODE_G) __stcs(dst, val);        // chunk buffer: streaming, as in the E epilogue
                else *dst = val;
              }
            }
          }
        } else {
          // fp32 outputs: 32 columns (128 bytes per row) per staging round; dW may accumulate
          float* obase = reinterpret_cast<float*>(p.out) + grow_warp0 * p.ldo;
#pragma unroll 1
          for (int ch = 0; ch < HALF_N / 32; ++ch) {
            const int col0 = col_half + ch * 32;
            if (col0 >= p.cols_valid) break;
            uint32_t v[32];
            tmem_ld32(taddr + ch * 32, v);
            if (MODE == MODE_DH && p.rowscale) {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(rs == 0.0f ? 0.0f : __uint_as_float(v[j]) * rs);
            }
            uint4 piece[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) piece[q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            stage_put(stage, lane, piece);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              int r, cc;
              const uint4 raw4 = stage_get(stage, lane, i, r, cc);
              if (grow_warp0 + r < p.rows_valid) {
                float* dst = obase + (int64_t)r * p.ldo + col0 + cc * 4;
                if (MODE == MODE_DW && p.n_shards > 0) {
                  // reduce-scatter form: this tile, plus the sum of the earlier chunks' tiles held in `out`,
                  // goes to the owner of the vocabulary row (its memory may be another GPU's: a plain
                  // peer store-reduction over NVLink, no load from there and nothing to wait for)
                  float4 val = make_float4(__uint_as_float(raw4.x), __uint_as_float(raw4.y), __uint_as_float(raw4.z),
                                           __uint_as_float(raw4.w));
                  if (p.accumulate) {
                    const float4 old = *reinterpret_cast<const float4*>(dst);
                    val.x += old.x; val.y += old.y; val.z += old.z; val.w += old.w;
                  }
                  const int64_t vrow = grow_warp0 + r;
                  const int owner = (int)(vrow / p.shard_rows);
                  float* sdst = p.shard[owner] + (vrow - (int64_t)owner * p.shard_rows) * p.ldo + col0 + cc * 4;
                  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                               ::"l"(sdst), "f"(val.x), "f"(val.y), "f"(val.z), "f"(val.w) : "memory");
                } else if (p.accumulate) {
                  // Added in L2, nothing comes back: no load latency in this (un-overlapped) epilogue.
                  // Each element receives exactly one addend per launch and launches are ordered on
                  // the stream, so the summation order is fixed.
                  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                               ::"l"(dst), "f"(__uint_as_float(raw4.x)), "f"(__uint_as_float(raw4.y)),
                                 "f"(__uint_as_float(raw4.z)), "f"(__uint_as_float(raw4.w))
                               : "memory");
                } else {
                  *reinterpret_cast<uint4*>(dst) = raw4;
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_leader);
      }
      if ((MODE == MODE_FWD || MODE == MODE_E) && ok && row_ok) {
        FwdPartial part;
        part.m2 = m2; part.l = l; part.zt = zt; part.pad = ez;
        p.partials[(int64_t)((u % p.nsplit) * 2 + half) * p.T + (grow - p.part_row0)] = part;
      }
    }
  }

  else if (warp == PACER_WARP && rank == 0 && p.progress != nullptr) {
    // ------------------------------------------------------------------ pacer (leader CTA)
    // Publishes this pair's k-block count, reads every pair's, and hands the producer its limit.  A
    // few loads and one sleep per turn; it ends when the producer has, or after kPacerMaxSpins turns
    // (then with the limit lifted, so that nobody waits for a pacer that has gone).
    volatile uint32_t* progress = p.progress;
    for (uint32_t spins = 0;; ++spins) {
      const uint32_t mine = *pace_mine;
      if (lane == 0) progress[group] = mine;
      if (mine == 0xFFFFFFFFu) break;
      if (spins >= kPacerMaxSpins) {
        if (lane == 0) { *pace_limit = 0xFFFFFFFFu; progress[group] = 0xFFFFFFFFu; }
        break;
      }
      // The slowest pair that is still within reach: one that is more than kLagCut windows behind this
      // pair (its CTAs started late because another kernel held their SMs, say) cannot share L2
      // lines with it any more, and waiting for it would only pass its delay on to everybody.
      const uint32_t reach = (uint32_t)kLagCut * (uint32_t)p.window;
      uint32_t mn = 0xFFFFFFFFu;
      for (int g = lane; g < n_groups; g += 32) {
        const uint32_t v = progress[g];
        if (v >= mine || mine - v <= reach) mn = min(mn, v);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      if (lane == 0) *pace_limit = (mn > 0xFFFFFFFFu - (uint32_t)p.window) ? 0xFFFFFFFFu : mn + (uint32_t)p.window;
      __nanosleep(kPacerSleepNs);
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {                       // let copies still in flight land before the CTA retires
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                       // the peer may still be reading this CTA's shared / tensor memory
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

// A wait that nothing ever satisfies, through the same bounded-wait routine the pipeline uses:
// checks that a stuck barrier ends in SPO_DEV_TIMEOUT and a clean return instead of a hang.
__global__ void bounded_wait_probe_kernel(int32_t* d_status, unsigned long long limit_ns, int* reached_end) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait<64>(smem_u32(&bar), 0, &abort_flag, d_status, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && reached_end) *reached_end = ok ? 2 : 1;
}

// ---------------------------------------------------------------------------
// host side: tensor maps and launches
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 2-D bf16 tensor [outer][inner] with row pitch `pitch_elems`; box = {64 inner, box_outer}; 128-byte swizzle;
// out-of-bounds elements read as zero.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint64_t pitch_elems, uint32_t box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {pitch_elems * 2};
  cuuint32_t box[2] = {64, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// How many k-blocks a CTA pair may run ahead of the slowest pair before it holds back.
#ifndef SPO_TUNE_WINDOW_SWEEP
#define SPO_TUNE_WINDOW_SWEEP 32
#endif
#ifndef SPO_TUNE_WINDOW_STREAM
#define SPO_TUNE_WINDOW_STREAM 16
#endif
constexpr int kWindowSweep = SPO_TUNE_WINDOW_SWEEP;
constexpr int kWindowStream = SPO_TUNE_WINDOW_STREAM;

// CTA pairs that can be resident at once (one CTA per SM).
int group_count() { return sm_count() / CG; }

// CTA pairs of this instantiation that can be resident together on a device (0 = not yet asked).
// The kernel is persistent and its pairs pace one another, so a grid must not exceed it.  One slot
// per device, filled once; concurrent first calls compute the same value (atomic stores).
template <int MODE, bool ENT>
cudaError_t resident_groups(int* out) {
  static std::atomic<int> cached[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int n = cached[dev].load(std::memory_order_acquire);
  if (n == 0) {
    e = cudaFuncSetAttribute(spo_gemm_kernel<MODE, ENT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t q = {};
    q.gridDim = dim3(group_count() * CG, 1, 1);
    q.blockDim = dim3(NUM_THREADS, 1, 1);
    q.dynamicSmemBytes = SMEM_BYTES;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = CG;
    qa[0].val.clusterDim.y = 1;
    qa[0].val.clusterDim.z = 1;
    q.attrs = qa;
    q.numAttrs = 1;
    e = cudaOccupancyMaxActiveClusters(&n, spo_gemm_kernel<MODE, ENT>, &q);
    if (e != cudaSuccess) return e;
    if (n < 1) return cudaErrorLaunchOutOfResources;
    if (n > group_count()) n = group_count();
    cached[dev].store(n, std::memory_order_release);
  }
  *out = n;
  return cudaSuccess;
}

template <int MODE, bool ENT = false>
cudaError_t launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmParams& p_in, uint32_t* progress,
                        cudaStream_t st) {
  int max_groups = 0;
  cudaError_t e0 = resident_groups<MODE, ENT>(&max_groups);
  if (e0 != cudaSuccess) return e0;
  const int units = p_in.m_tiles * p_in.nsplit;
  if (units <= 0) return cudaSuccess;
  GemmParams p = p_in;
  // k-blocks a pair may run ahead of the slowest one.  E / FWD / G sweep short tiles (d / 64 k-blocks) and
  // re-read their row strip per tile; dH / dW stream both operands through one long tile.
  p.window = (MODE == MODE_DH || MODE == MODE_DW) ? kWindowStream : kWindowSweep;
  p.progress = nullptr;
  if (p.window > 0 && progress) {
    cudaError_t e = cudaMemsetAsync(progress, 0, kProgressBytes, st);
    if (e != cudaSuccess) return e;
    p.progress = progress;
  }
  const int groups = units < max_groups ? units : max_groups;
  if ((size_t)groups * 4 > kProgressBytes) p.progress = nullptr;       // more pairs than progress words: run unpaced
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(groups * CG, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, spo_gemm_kernel<MODE, ENT>, a, b, p);
}

// Operand box heights (rows per TMA box) for K-major operands.
constexpr uint32_t kBoxA = BM;
constexpr uint32_t kBoxB = BSUB_ROWS;

// How many splits of the column tiles a FWD / G launch uses.  All pairs running at one time form
// a rectangle of (pairs / nsplit) row tiles x nsplit column positions; per sweep step L2 has to hold
// that many A tiles (re-read every step) plus nsplit B tiles (streamed).  Fewer splits mean fewer
// re-reads of W from HBM; the choice also avoids a short last split (pairs would fall out of step)
// and a nearly empty last round of units.
int pick_fwd_split(int64_t m_tiles, int n_tiles, int d) {
#ifdef SPO_TUNE_NSPLIT
  if (m_tiles > 8) return SPO_TUNE_NSPLIT < n_tiles ? SPO_TUNE_NSPLIT : n_tiles;
#endif
  const int groups = group_count();
  const double a_tile = (double)GROUP_M * d * 2, b_tile = (double)BN * d * 2;
  const double l2_budget = 56e6;
  int best = 1;
  double best_score = -1.0;
  for (int ns = 1; ns <= n_tiles && ns <= 256; ++ns) {
    const int per = (int)ceil_div(n_tiles, ns);
    if ((int)ceil_div(n_tiles, per) != ns) continue;               // not a distinct partition
    const double ragged = (double)(ns * per - n_tiles) / (double)(ns * per);
    const int64_t units = m_tiles * ns;
    const int64_t rounds = ceil_div(units, groups);
    const double fill = (double)units / (double)(rounds * groups);
    const double rows_live = (double)(m_tiles < (groups + ns - 1) / ns ? m_tiles : (groups + ns - 1) / ns);
    const double footprint = rows_live * a_tile + ns * b_tile;
    double score = fill * (1.0 - ragged) / (1.0 + 0.01 * ns);
    if (footprint > l2_budget) score *= l2_budget / footprint;
    if (score > best_score) { best_score = score; best = ns; }
  }
  return best;
}

// Splits of the vocabulary tiles actually used for a given shape.
int fwd_unit_splits(int64_t T, int32_t d, int32_t V) {
  const int64_t m_tiles = ceil_div(T, GROUP_M);
  const int n_tiles = (int)ceil_div(V, BN);
  return pick_fwd_split(m_tiles, n_tiles, d);
}

}  // namespace

// Number of forward partials per token row (two column halves per vocabulary split);
// the workspace layout depends on it.
int fwd_bf16_nsplit(int64_t T, int32_t d, int32_t V) { return 2 * fwd_unit_splits(T, d, V); }

cudaError_t launch_fwd_bf16(const void* H, const void* W, const int32_t* y, int64_t T, int32_t d, int32_t V,
                            FwdPartial* partials, int nsplit, int want_entropy, uint32_t* progress, int32_t* d_status,
                            cudaStream_t st) {
  if (T == 0) return cudaSuccess;
  CUtensorMap ma, mb;
  if (!make_map(&ma, H, d, T, d, kBoxA) || !make_map(&mb, W, d, V, d, kBoxB)) return cudaErrorInvalidValue;
  GemmParams p{};
  p.m_tiles = (int)ceil_div(T, GROUP_M);
  p.n_tiles = (int)ceil_div(V, BN);
  p.nsplit = nsplit / 2;
  p.per_split = (int)ceil_div(p.n_tiles, p.nsplit);
  p.k_blocks = (int)ceil_div(d, BK);
  p.rows_valid = T;
  p.cols_valid = V;
  p.out_row0 = 0;
  p.y = y;
  p.partials = partials;
  p.T = T;
  p.d_status = d_status;
  if (want_entropy) return launch_gemm<MODE_FWD, true>(ma, mb, p, progress, st);
  return launch_gemm<MODE_FWD>(ma, mb, p, progress, st);
}

BwdWs bwd_ws_layout(int64_t T, int32_t d, int32_t V) {
  BwdWs L{};
  // Token rows per chunk: half as many row tiles as there are CTA pairs.  With d/512 column
  // tiles (a multiple of 2 for the usual hidden sizes) the dH tiles of a full chunk then fill the
  // pairs a whole number of times, and the chunk buffer stays at a few GB.
  const int groups = group_count();
  int64_t m_tiles = groups / 2 > 0 ? groups / 2 : 1;
  int64_t rows = m_tiles * GROUP_M;
  const int64_t t_pad = ceil_div(T > 0 ? T : 1, GROUP_M) * GROUP_M;
  if (rows > t_pad) rows = t_pad;
  L.chunk_rows = rows;
  L.ldg = ceil_div(V, BN) * BN;
  L.g = 0;
  L.progress = align_up((size_t)rows * (size_t)L.ldg * 2, 256);
  L.total = L.progress + kProgressBytes;
  return L;
}

namespace {

// dH rows [t0, t0 + rows) = G W, where G is the chunk buffer (one-pass path: times `rowscale`, indexed by
// token row, in the epilogue).
cudaError_t launch_dh(const CUtensorMap& mG_k, const CUtensorMap& mW_mn, int64_t t0, int64_t rows, int64_t T,
                      int32_t d, int32_t V, void* dH, int32_t dH_dtype, const float* rowscale, uint32_t* progress,
                      int32_t* d_status, cudaStream_t st) {
  const int n_tiles_d = (int)ceil_div(d, BN);
  GemmParams p{};
  p.m_tiles = (int)ceil_div(rows, GROUP_M);
  p.n_tiles = n_tiles_d;
  p.nsplit = n_tiles_d;
  p.per_split = 1;
  p.k_blocks = (int)ceil_div(V, BK);
  p.rows_valid = T;
  p.cols_valid = d;
  p.out_row0 = t0;
  p.out = dH; p.out_bf16 = (dH_dtype == SPO_DTYPE_BF16); p.ldo = d; p.accumulate = 0;
  p.rowscale = rowscale;
  p.d_status = d_status;
  return launch_gemm<MODE_DH>(mG_k, mW_mn, p, progress, st);
}

// dW (+)= G^T Hk over `rows` token rows: G is the chunk buffer read as an M-major operand, Hk the
// matching rows of the hidden states (read from row `h_row0` of their tensor map).  `tile0`, `tiles`:
// the slab of 256-row vocabulary tiles this launch covers (the whole vocabulary: 0, all of them).
cudaError_t launch_dw(const CUtensorMap& mG_mn, const CUtensorMap& mH_mn, int64_t h_row0, int64_t rows, int32_t d,
                      int32_t V, float* dW, int dw_accumulate, int tile0, int tiles, uint32_t* progress,
                      int32_t* d_status, cudaStream_t st, const spo_dw_shards* shards = nullptr) {
  const int n_tiles_d = (int)ceil_div(d, BN);
  GemmParams p{};
  p.m_tiles = tiles;
  p.m_tile0 = tile0;
  p.n_tiles = n_tiles_d;
  p.nsplit = n_tiles_d;
  p.per_split = 1;
  p.k_blocks = (int)ceil_div(rows, BK);
  p.b_k0 = (int)h_row0;
  p.rows_valid = V;
  p.cols_valid = d;
  p.out_row0 = 0;
  p.out = dW; p.out_bf16 = 0; p.ldo = d; p.accumulate = dw_accumulate;
  if (shards) {
    p.n_shards = shards->n_shards;
    p.shard_rows = shards->rows_per_shard;
    for (int k = 0; k < shards->n_shards; ++k) p.shard[k] = shards->shard[k];
  }
  p.d_status = d_status;
  return launch_gemm<MODE_DW>(mG_mn, mH_mn, p, progress, st);
}

}  // namespace

cudaError_t launch_bwd_bf16(const void* H, const void* W, const int32_t* y, const float* lse,
                            const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V,
                            void* dH, int32_t dH_dtype, float* dW, int accumulate,
                            char* ws, const BwdWs& L, int32_t* d_status, cudaStream_t st) {
  __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(ws + L.g);
  uint32_t* progress = reinterpret_cast<uint32_t*>(ws + L.progress);
  if (T == 0) {
    if (!accumulate) return cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)V * d, st);
    return cudaSuccess;
  }
  CUtensorMap mH_k, mW_k, mW_mn, mH_mn;
  if (!make_map(&mH_k, H, d, T, d, kBoxA) || !make_map(&mW_k, W, d, V, d, kBoxB) ||
      !make_map(&mW_mn, W, d, V, d, 64) || !make_map(&mH_mn, H, d, T, d, 64))
    return cudaErrorInvalidValue;
  const int n_tiles_v = (int)ceil_div(V, BN);
  cudaError_t e;
  int chunk = 0;
  for (int64_t t0 = 0; t0 < T; t0 += L.chunk_rows, ++chunk) {
    const int64_t rows = (T - t0) < L.chunk_rows ? (T - t0) : L.chunk_rows;
    const int m_tiles = (int)ceil_div(rows, GROUP_M);
    CUtensorMap mG_k, mG_mn;
    if (!make_map(&mG_k, G, V, rows, L.ldg, kBoxA) || !make_map(&mG_mn, G, V, rows, L.ldg, 64))
      return cudaErrorInvalidValue;
    // 1) logits of the chunk, rewritten in place as g (bf16)
    {
      GemmParams p{};
      p.m_tiles = m_tiles;
      p.n_tiles = n_tiles_v;
      p.nsplit = pick_fwd_split(m_tiles, n_tiles_v, d);
      p.per_split = (int)ceil_div(n_tiles_v, p.nsplit);
      p.k_blocks = (int)ceil_div(d, BK);
      p.a_row0 = (int)t0;
      p.rows_valid = T;
      p.cols_valid = V;
      p.out_row0 = t0;
      p.y = y; p.lse = lse; p.coef = coef; p.grad_loss = grad_loss;
      p.T = T;
      p.G = G; p.ldg = L.ldg;
      p.d_status = d_status;
      if ((e = launch_gemm<MODE_G>(mH_k, mW_k, p, progress, st)) != cudaSuccess) return e;
    }
    // 2) dH rows of the chunk = G W;  3) dW (+)= G^T H_chunk
    if ((e = launch_dh(mG_k, mW_mn, t0, rows, T, d, V, dH, dH_dtype, nullptr, progress, d_status, st)) != cudaSuccess)
      return e;
    if ((e = launch_dw(mG_mn, mH_mn, t0, rows, d, V, dW, (accumulate || chunk > 0) ? 1 : 0, 0,
                       (int)ceil_div(V, GROUP_M), progress, d_status, st)) != cudaSuccess)
      return e;
  }
  return cudaSuccess;
}

// ---------------------------------------------------------------------------
// One-pass forward+backward: three contractions per token instead of the four of
// forward-then-backward.
//   PRE      the logits of the first vocabulary tile for all rows (0.3 % of one contraction): their
//            row maxima fix every row's reference exponent
//   per chunk c of token rows, into slot c % slots of the chunk buffers:
//     E(c)     logits contraction; epilogue: sum of exponentials, target logit, e = 2^(z log2e - ref) as bf16
//     fin(c)   lse, logp, ratio, surrogate, coef, loss terms; row scale; the target entry of e patched
//     scale(c) the chunk's rows of H times their row scale (bf16), the operand of the dW contraction
//     DH(c)    dH rows = rowscale * (e W)
//   per group of `slots` chunks:  DW   dW (+)= e^T (rowscale H) over the rows of the whole group
// Contracting dW over several chunks at once divides its read-modify-write passes over the
// [V x d] fp32 matrix (and its accumulator drains) by that number.
// ---------------------------------------------------------------------------
#ifndef SPO_DW_CHUNK_GROUP
#define SPO_DW_CHUNK_GROUP 2
#endif
constexpr int kDwChunkGroup = SPO_DW_CHUNK_GROUP;

FusedWs fused_ws_layout(int64_t T, int32_t d, int32_t V, int32_t S) {
  FusedWs L{};
  const BwdWs b = bwd_ws_layout(T, d, V);
  L.chunk_rows = b.chunk_rows;
  L.ldg = b.ldg;
  const int n_tiles_v = (int)ceil_div(V, BN);
  const int64_t t_eff = T > 0 ? T : 1;
  const int64_t n_chunks = ceil_div(t_eff, L.chunk_rows);
  L.slots = (int)(n_chunks < kDwChunkGroup ? n_chunks : kDwChunkGroup);
  // partials: the full chunk and the (shorter) last chunk may pick different split counts
  const int64_t full_rows = t_eff < L.chunk_rows ? ceil_div(t_eff, GROUP_M) * GROUP_M : L.chunk_rows;
  size_t part_elems = (size_t)2 * pick_fwd_split(full_rows / GROUP_M, n_tiles_v, d) * (size_t)full_rows;
  const int64_t tail = t_eff % L.chunk_rows;
  if (t_eff > L.chunk_rows && tail > 0) {
    const int64_t tail_rows = ceil_div(tail, GROUP_M) * GROUP_M;
    const size_t e2 = (size_t)2 * pick_fwd_split(tail_rows / GROUP_M, n_tiles_v, d) * (size_t)tail_rows;
    if (e2 > part_elems) part_elems = e2;
  }
  L.fin_blocks = ceil_div(t_eff, kFinalizeThreads);
  size_t off = 0;
  L.g = off;          off = align_up(off + (size_t)L.slots * (size_t)L.chunk_rows * (size_t)L.ldg * 2, 256);
  L.hs = off;         off = align_up(off + (size_t)L.slots * (size_t)L.chunk_rows * (size_t)d * 2, 256);
  L.pre = off;        off = align_up(off + sizeof(FwdPartial) * 2 * (size_t)t_eff, 256);
  L.rowscale = off;   off = align_up(off + sizeof(float) * (size_t)t_eff, 256);
  L.partials = off;   off = align_up(off + sizeof(FwdPartial) * part_elems, 256);
  L.progress = off;   off = align_up(off + kProgressBytes, 256);
  L.block_sums = off; off = align_up(off + sizeof(double) * (size_t)L.fin_blocks, 256);
  L.counters = off;   off = align_up(off + 4 * sizeof(int32_t), 256);
  L.seq_cnt = off;    off = align_up(off + sizeof(int32_t) * (size_t)(S > 0 ? S : 1), 256);
  L.total = off;
  return L;
}

namespace {
// Row tiles (of GROUP_M vocabulary rows) per slab: whole rounds of units, so that no slab ends on a
// partly filled round of CTA pairs.
int slab_tiles(int32_t V, int32_t d, int n_wanted, int* n_out) {
  const int tiles = (int)ceil_div(V, GROUP_M), n_tiles_d = (int)ceil_div(d, BN), groups = group_count();
  int g = groups, b = n_tiles_d;                       // gcd
  while (b) { const int t = g % b; g = b; b = t; }
  const int quantum = groups / g;                      // row tiles whose units fill the pairs a whole number of times
  if (n_wanted < 1) n_wanted = 1;
  int per = tiles / n_wanted / quantum * quantum;      // rounded down: the last slab takes what is left over
  if (per < quantum) per = quantum;
  const int n = (int)ceil_div(tiles, per);
  *n_out = n < n_wanted ? n : n_wanted;
  return per;
}
}  // namespace

int dw_slab_rows(int32_t V, int32_t d, int n_wanted, int64_t* row_begin) {
  int n = 1;
  const int per = slab_tiles(V, d, n_wanted, &n);
  for (int k = 0; k < n; ++k) row_begin[k] = (int64_t)k * per * GROUP_M;
  row_begin[n] = V;                                    // slab n-1 runs to the end of the vocabulary
  return n;
}

cudaError_t launch_fused_bf16(const FusedArgs& a, char* ws, const FusedWs& L, cudaStream_t st) {
  FwdPartial* partials = reinterpret_cast<FwdPartial*>(ws + L.partials);
  FwdPartial* pre = reinterpret_cast<FwdPartial*>(ws + L.pre);
  float* rowscale = reinterpret_cast<float*>(ws + L.rowscale);
  uint32_t* progress = reinterpret_cast<uint32_t*>(ws + L.progress);
  double* block_sums = reinterpret_cast<double*>(ws + L.block_sums);
  int32_t* counters = reinterpret_cast<int32_t*>(ws + L.counters);
  int32_t* seq_cnt = reinterpret_cast<int32_t*>(ws + L.seq_cnt);
  __nv_bfloat16* gbuf = reinterpret_cast<__nv_bfloat16*>(ws + L.g);
  __nv_bfloat16* hsbuf = reinterpret_cast<__nv_bfloat16*>(ws + L.hs);
  const spo_params& pr = *a.params;
  const int64_t T = a.T;
  const int32_t d = a.d, V = a.V;
  cudaError_t e = launch_fwd_prepare(a.mask, T, a.cu_seqlens, a.S, pr.agg_mode != 0, seq_cnt, counters, st);
  if (e != cudaSuccess) return e;
  if (T == 0) {
    e = launch_fwd_finalize(partials, 0, a.y, a.logp_old, a.mask, a.cu_seqlens, a.a_norm, 0, V, a.S, a.loss, a.logp,
                            a.lse, a.coef, a.seq_sums, a.entropy, block_sums, counters, seq_cnt, pr, L.fin_blocks,
                            a.d_status, st);
    if (e != cudaSuccess) return e;
    if (!a.accumulate && (e = cudaMemsetAsync(a.dW, 0, sizeof(float) * (size_t)V * d, st)) != cudaSuccess) return e;
    if (a.shards && a.accumulate && (e = launch_dw_scatter_add(a.dW, V, d, *a.shards, st)) != cudaSuccess) return e;
    if (a.n_slabs > 0 && a.events) {              // nothing to contract: every slab is final at once
      int n = 1;
      slab_tiles(V, d, a.n_slabs, &n);
      for (int k = 0; k < n; ++k)
        if ((e = cudaEventRecord(a.events[k], st)) != cudaSuccess) return e;
    }
    return cudaSuccess;
  }
  CUtensorMap mH_k, mW_k, mW_mn;
  if (!make_map(&mH_k, a.H, d, T, d, kBoxA) || !make_map(&mW_k, a.W, d, V, d, kBoxB) ||
      !make_map(&mW_mn, a.W, d, V, d, 64))
    return cudaErrorInvalidValue;
  const int n_tiles_v = (int)ceil_div(V, BN);
  const int n_chunks = (int)ceil_div(T, L.chunk_rows);
  const bool ent = a.entropy != nullptr;

  // PRE: first vocabulary tile of every row (the forward's kernel on one column tile)
  {
    GemmParams p{};
    p.m_tiles = (int)ceil_div(T, GROUP_M);
    p.n_tiles = 1;
    p.nsplit = 1;
    p.per_split = 1;
    p.k_blocks = (int)ceil_div(d, BK);
    p.rows_valid = T;
    p.cols_valid = V;
    p.y = a.y;
    p.partials = pre;
    p.T = T;
    p.d_status = a.d_status;
    if ((e = launch_gemm<MODE_FWD>(mH_k, mW_k, p, progress, st)) != cudaSuccess) return e;
  }

  for (int c0 = 0; c0 < n_chunks; c0 += L.slots) {
    int64_t group_rows = 0;
    for (int c = c0; c < n_chunks && c < c0 + L.slots; ++c) {
      const int slot = c - c0;
      const int64_t t0 = (int64_t)c * L.chunk_rows;
      const int64_t rows = (T - t0) < L.chunk_rows ? (T - t0) : L.chunk_rows;
      const int m_tiles = (int)ceil_div(rows, GROUP_M);
      const int64_t rows_pad = (int64_t)m_tiles * GROUP_M;
      __nv_bfloat16* G = gbuf + (size_t)slot * (size_t)L.chunk_rows * (size_t)L.ldg;
      // E: logits of chunk c
      const int nsplit = pick_fwd_split(m_tiles, n_tiles_v, d);
      {
        GemmParams p{};
        p.m_tiles = m_tiles;
        p.n_tiles = n_tiles_v;
        p.nsplit = nsplit;
        p.per_split = (int)ceil_div(n_tiles_v, p.nsplit);
        p.k_blocks = (int)ceil_div(d, BK);
        p.a_row0 = (int)t0;
        p.rows_valid = T;
        p.cols_valid = V;
        p.out_row0 = t0;
        p.y = a.y;
        p.partials = partials;
        p.T = rows_pad;
        p.part_row0 = t0;
        p.G = G; p.ldg = L.ldg;
        p.pre = pre; p.pre_ld = T;
        p.d_status = a.d_status;
        e = ent ? launch_gemm<MODE_E, true>(mH_k, mW_k, p, progress, st)
                : launch_gemm<MODE_E, false>(mH_k, mW_k, p, progress, st);
        if (e != cudaSuccess) return e;
      }
      // fin: per-token outputs of chunk c's rows, loss terms per block, row scale, patched target entries
      {
        FinalizeRange rg;
        rg.t_begin = t0;
        rg.part_ld = rows_pad;
        rg.block0 = (int)(t0 / kFinalizeThreads);
        rg.total_blocks = (int)L.fin_blocks;
        rg.last = (c == n_chunks - 1) ? 1 : 0;
        OnePassFix fix;
        fix.G = reinterpret_cast<uint16_t*>(G);
        fix.ldg = L.ldg;
        fix.g_row0 = t0;
        fix.rowscale = rowscale;
        fix.grad_loss = a.grad_loss;
        e = launch_fwd_finalize(partials, 2 * nsplit, a.y, a.logp_old, a.mask, a.cu_seqlens, a.a_norm, t0 + rows, V,
                                a.S, a.loss, a.logp, a.lse, a.coef, a.seq_sums, a.entropy, block_sums, counters, seq_cnt,
                                pr, L.fin_blocks, a.d_status, st, &rg, &fix);
        if (e != cudaSuccess) return e;
      }
      // the chunk's rows of H times their row scale, behind the rows of the group's earlier chunks
      e = launch_scale_rows(a.H, rowscale, t0, rows, d * 2, hsbuf + (size_t)slot * (size_t)L.chunk_rows * (size_t)d, st);
      if (e != cudaSuccess) return e;
      // DH: rows of chunk c
      {
        CUtensorMap mG_k;
        if (!make_map(&mG_k, G, V, rows, L.ldg, kBoxA)) return cudaErrorInvalidValue;
        e = launch_dh(mG_k, mW_mn, t0, rows, T, d, V, a.dH, a.dH_dtype, rowscale, progress, a.d_status, st);
        if (e != cudaSuccess) return e;
      }
      group_rows += rows;        // only the group's last chunk can be short, so the rows stay contiguous
    }
    // DW over the group's rows
    CUtensorMap mG_mn, mHs_mn;
    if (!make_map(&mG_mn, gbuf, V, group_rows, L.ldg, 64) || !make_map(&mHs_mn, hsbuf, d, group_rows, d, 64))
      return cudaErrorInvalidValue;
    const int tiles = (int)ceil_div(V, GROUP_M);
    const int dw_acc = (a.accumulate || c0 > 0) ? 1 : 0;
    if (a.n_slabs > 0 && a.events && c0 + L.slots >= n_chunks) {
      // the last contraction of dW, slab by slab: behind each slab its rows are final
      int n = 1;
      const int per = slab_tiles(V, d, a.n_slabs, &n);
      for (int k = 0; k < n; ++k) {
        const int t_begin = k * per, t_count = k == n - 1 ? tiles - t_begin : per;
        e = launch_dw(mG_mn, mHs_mn, 0, group_rows, d, V, a.dW, dw_acc, t_begin, t_count, progress, a.d_status, st);
        if (e != cudaSuccess) return e;
        if ((e = cudaEventRecord(a.events[k], st)) != cudaSuccess) return e;
      }
    } else {
      // reduce-scatter form: the call's last contraction sends the finished tiles to their owners
      const spo_dw_shards* sh = (a.shards && c0 + L.slots >= n_chunks) ? a.shards : nullptr;
      e = launch_dw(mG_mn, mHs_mn, 0, group_rows, d, V, a.dW, dw_acc, 0, tiles, progress, a.d_status, st, sh);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

cudaError_t launch_bounded_wait_probe(int32_t* d_status, uint32_t limit_us, int32_t* reached_end, cudaStream_t st) {
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(d_status, (unsigned long long)limit_us * 1000ull, reached_end);
  return cudaGetLastError();
}

}  // namespace spo
