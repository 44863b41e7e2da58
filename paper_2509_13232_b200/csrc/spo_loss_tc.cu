// bf16 loss forward / backward on the 5th-generation tensor cores (sm_100a).
//
// One persistent, warp-specialised kernel template does every contraction of the path:
//   FWD : S = H W^T tile by tile; epilogue keeps an online (max, sum-exp, target logit)
//         per token row in registers across the vocabulary tiles of its split.
//   G   : the same contraction for one chunk of token rows; epilogue turns each logit
//         into g = c_t (1[v=y_t] - e^{z-lse_t}) and writes it as bf16 into the chunk buffer.
//   DH  : dH_chunk = G W        (A = G, K-major;  B = W read as an N-major operand)
//   DW  : dW (+)= G^T H_chunk   (A = G read as an M-major operand; B = H, N-major)
//
// Pipeline per CTA (one CTA per SM, 192 threads):
//   warp 0 : allocates tensor memory; lane 0 issues the TMA loads (128-byte swizzle)
//            into a 4-stage shared-memory ring, signalling "full" mbarriers.
//   warp 1 : lane 0 issues tcgen05.mma (128x256x16, bf16 -> fp32) into one of two
//            256-column accumulators in tensor memory; tcgen05.commit releases the
//            stage ("empty") and, after the last k-block, publishes the accumulator.
//   warps 2-5 : epilogue; each owns the 32 accumulator lanes its warp id selects,
//            reads them with tcgen05.ld and applies the mode's fused epilogue while
//            the next tile accumulates in the other buffer.
// Every mbarrier wait is bounded: when it runs out the CTA raises SPO_DEV_TIMEOUT,
// all roles leave their loops, tensor memory is released and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "spo_internal.h"

namespace spo {

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
constexpr unsigned long long kWaitLimitNs = 4000000000ull;

constexpr float kLog2e = 1.4426950408889634f;

enum : int { MODE_FWD = 0, MODE_G = 1, MODE_DH = 2, MODE_DW = 3 };

struct GemmParams {
  int m_tiles, n_tiles, nsplit, per_split;   // work decomposition: unit = (m tile, split of the n tiles)
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
  int64_t T;
  __nv_bfloat16* G;
  int64_t ldg;
  // DH / DW
  void* out;
  int out_bf16;
  int64_t ldo;
  int accumulate;
  int32_t* d_status;
};

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* d_status) {
  uint32_t spins = 0;
  unsigned long long t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      unsigned long long now = global_timer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        if (d_status) atomicOr(d_status, SPO_DEV_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
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
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
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

// Instruction descriptor for kind::f16: fp32 accumulate, bf16 A and B, M = 128, N = 256.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

struct Unit { int m_tile, n_begin, n_end; };
__device__ __forceinline__ Unit unit_of(int u, const GemmParams& p) {
  Unit r;
  const int split = u % p.nsplit;
  r.m_tile = u / p.nsplit;
  r.n_begin = split * p.per_split;
  r.n_end = min(r.n_begin + p.per_split, p.n_tiles);
  return r;
}

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
spo_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  constexpr bool A_MN = (MODE == MODE_DW);
  constexpr bool B_MN = (MODE == MODE_DH || MODE == MODE_DW);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bars = base + STAGES * STAGE_BYTES;
  const uint32_t full0 = bars, empty0 = bars + 8 * STAGES, tfull0 = bars + 16 * STAGES, tempty0 = tfull0 + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + STAGES * STAGE_BYTES + 16 * STAGES + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + STAGES * STAGE_BYTES + 16 * STAGES + 40);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_units = p.m_tiles * p.nsplit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const Unit un = unit_of(u, p);
        for (int n = un.n_begin; n < un.n_end && ok; ++n) {
          for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag, p.d_status)) { ok = false; break; }
            const uint32_t fb = full0 + 8 * s;
            const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
            mbar_expect_tx(fb, STAGE_BYTES);
            if (!A_MN) {
              tma_load_2d(sa, &tmA, kb * BK, p.a_row0 + un.m_tile * BM, fb);
            } else {
#pragma unroll
              for (int b = 0; b < BM / 64; ++b)
                tma_load_2d(sa + b * 8192, &tmA, un.m_tile * BM + b * 64, p.a_row0 + kb * BK, fb);
            }
            if (!B_MN) {
              tma_load_2d(sb, &tmB, kb * BK, n * BN, fb);
            } else {
#pragma unroll
              for (int b = 0; b < BN / 64; ++b)
                tma_load_2d(sb + b * 8192, &tmB, n * BN + b * 64, p.b_k0 + kb * BK, fb);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(A_MN, B_MN);
      uint32_t it = 0, tile = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const Unit un = unit_of(u, p);
        for (int n = un.n_begin; n < un.n_end && ok; ++n, ++tile) {
          const uint32_t acc = tile & 1u, aph = (tile >> 1) & 1u;
          if (!mbar_wait(tempty0 + 8 * acc, aph ^ 1u, abort_flag, p.d_status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + acc * BN;
          for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.d_status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
            for (int j = 0; j < BK / 16; ++j) {
              const uint64_t da = A_MN ? smem_desc(sa + j * 2048, 8192, 1024) : smem_desc(sa + j * 32, 16, 1024);
              const uint64_t db = B_MN ? smem_desc(sb + j * 2048, 8192, 1024) : smem_desc(sb + j * 32, 16, 1024);
              umma_bf16(tmem_d, da, db, idesc, (kb | j) != 0 ? 1u : 0u);
            }
            umma_commit(empty0 + 8 * s);
          }
          if (ok) umma_commit(tfull0 + 8 * acc);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;                    // tensor-memory lanes this warp may read
    const int row = quarter * 32 + lane;             // row of the 128-row tile
    uint32_t tile = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
      const Unit un = unit_of(u, p);
      const int64_t grow = p.out_row0 + (int64_t)un.m_tile * BM + row;   // global output row
      const bool row_ok = grow < p.rows_valid;
      // per-row state
      float m2 = -CUDART_INF_F, l = 0.0f, zt = -CUDART_INF_F;             // FWD
      int32_t yt = -1;
      float c = 0.0f, lse2 = 0.0f;                                         // G
      if (MODE == MODE_FWD || MODE == MODE_G) {
        if (row_ok) yt = p.y[grow];
        if (MODE == MODE_G && row_ok) { c = p.grad_loss * p.coef[grow]; lse2 = p.lse[grow] * kLog2e; }
      }
      for (int n = un.n_begin; n < un.n_end && ok; ++n, ++tile) {
        const uint32_t acc = tile & 1u, aph = (tile >> 1) & 1u;
        if (!mbar_wait(tfull0 + 8 * acc, aph, abort_flag, p.d_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
        const int col_tile = n * BN;
#pragma unroll 1
        for (int ch = 0; ch < BN / 32; ++ch) {
          const int col0 = col_tile + ch * 32;
          if (col0 >= p.cols_valid && MODE != MODE_G) break;          // nothing valid further right
          uint32_t v[32];
          tmem_ld32(taddr + ch * 32, v);
          if (MODE == MODE_FWD) {
            const bool tail = col0 + 32 > p.cols_valid;
            float cmax = -CUDART_INF_F;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              float z = __uint_as_float(v[j]);
              if (tail && col0 + j >= p.cols_valid) { z = -CUDART_INF_F; v[j] = __float_as_uint(z); }
              cmax = fmaxf(cmax, z);
            }
            const float mn = fmaxf(m2, cmax * kLog2e);
            float sum = 0.0f;
#pragma unroll
            for (int j = 0; j < 32; ++j) sum += exp2f(fmaf(__uint_as_float(v[j]), kLog2e, -mn));
            l = l * exp2f(m2 - mn) + sum;
            m2 = mn;
            if (yt >= col0 && yt < col0 + 32) {
              const int jj = yt - col0;
#pragma unroll
              for (int j = 0; j < 32; ++j) if (j == jj) zt = __uint_as_float(v[j]);
            }
          } else if (MODE == MODE_G) {
            if (row_ok) {
              uint32_t o[16];
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                float g0 = 0.0f, g1 = 0.0f;
                if (c != 0.0f) {
                  const float p0 = exp2f(fmaf(__uint_as_float(v[j]), kLog2e, -lse2));
                  const float p1 = exp2f(fmaf(__uint_as_float(v[j + 1]), kLog2e, -lse2));
                  g0 = c * ((col0 + j == yt ? 1.0f : 0.0f) - p0);
                  g1 = c * ((col0 + j + 1 == yt ? 1.0f : 0.0f) - p1);
                }
                if (col0 + j >= p.cols_valid) g0 = 0.0f;
                if (col0 + j + 1 >= p.cols_valid) g1 = 0.0f;
                o[j >> 1] = pack_bf16(g0, g1);
              }
              uint4* dst = reinterpret_cast<uint4*>(p.G + ((int64_t)un.m_tile * BM + row) * p.ldg + col0);
#pragma unroll
              for (int q = 0; q < 4; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
            }
          } else {
            if (row_ok) {
              if (p.out_bf16) {
                uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + grow * p.ldo + col0);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  dst[q] = make_uint4(pack_bf16(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])),
                                      pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                      pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                      pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
              } else {
                float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + grow * p.ldo + col0);
                if (p.accumulate) {
#pragma unroll
                  for (int q = 0; q < 8; ++q) {
                    float4 old = dst[q];
                    old.x += __uint_as_float(v[4 * q + 0]); old.y += __uint_as_float(v[4 * q + 1]);
                    old.z += __uint_as_float(v[4 * q + 2]); old.w += __uint_as_float(v[4 * q + 3]);
                    dst[q] = old;
                  }
                } else {
#pragma unroll
                  for (int q = 0; q < 8; ++q)
                    dst[q] = make_float4(__uint_as_float(v[4 * q + 0]), __uint_as_float(v[4 * q + 1]),
                                         __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      }
      if (MODE == MODE_FWD && ok && row_ok) {
        FwdPartial part;
        part.m2 = m2; part.l = l; part.zt = zt; part.pad = 0.0f;
        p.partials[(int64_t)(u % p.nsplit) * p.T + grow] = part;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {                       // let copies still in flight land before the CTA retires
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
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

template <int MODE>
cudaError_t launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmParams& p, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(spo_gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int units = p.m_tiles * p.nsplit;
  if (units <= 0) return cudaSuccess;
  const int grid = units < sm_count() ? units : sm_count();
  spo_gemm_kernel<MODE><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(a, b, p);
  return cudaGetLastError();
}

int pick_fwd_split(int64_t m_tiles, int n_tiles) {
  // Enough units to fill the machine, and several splits so that CTAs running together
  // share token tiles (which then stay in L2) while sweeping different parts of W.
  int sms = sm_count();
  int nsplit = 4;
  while (m_tiles * nsplit < 2 * (int64_t)sms && nsplit < n_tiles) nsplit *= 2;
  if (nsplit > n_tiles) nsplit = n_tiles;
  if (nsplit < 1) nsplit = 1;
  return nsplit;
}

}  // namespace

// nsplit used by the forward for a given shape (the workspace layout depends on it).
int fwd_bf16_nsplit(int64_t T, int32_t V) {
  const int64_t m_tiles = ceil_div(T, BM);
  const int n_tiles = (int)ceil_div(V, BN);
  int nsplit = pick_fwd_split(m_tiles, n_tiles);
  const int per = (int)ceil_div(n_tiles, nsplit);
  return (int)ceil_div(n_tiles, per);
}

cudaError_t launch_fwd_bf16(const void* H, const void* W, const int32_t* y, int64_t T, int32_t d, int32_t V,
                            FwdPartial* partials, int nsplit, int32_t* d_status, cudaStream_t st) {
  if (T == 0) return cudaSuccess;
  CUtensorMap ma, mb;
  if (!make_map(&ma, H, d, T, d, BM) || !make_map(&mb, W, d, V, d, BN)) return cudaErrorInvalidValue;
  GemmParams p{};
  p.m_tiles = (int)ceil_div(T, BM);
  p.n_tiles = (int)ceil_div(V, BN);
  p.per_split = (int)ceil_div(p.n_tiles, nsplit);
  p.nsplit = nsplit;
  p.k_blocks = (int)ceil_div(d, BK);
  p.rows_valid = T;
  p.cols_valid = V;
  p.out_row0 = 0;
  p.y = y;
  p.partials = partials;
  p.T = T;
  p.d_status = d_status;
  return launch_gemm<MODE_FWD>(ma, mb, p, st);
}

BwdWs bwd_ws_layout(int64_t T, int32_t d, int32_t V) {
  BwdWs L{};
  // Token rows per chunk: a multiple of 128 chosen so that the dH tiles of a full chunk
  // (row tiles x d/256 column tiles) fill the SMs a whole number of times.
  const int sms = sm_count();
  const int n_tiles_d = (int)ceil_div(d, BN);
  int64_t m_tiles = 32;
  for (int64_t cand = 24; cand <= 64; ++cand)
    if ((cand * n_tiles_d) % sms == 0) { m_tiles = cand; break; }
  int64_t rows = m_tiles * BM;
  const int64_t t_pad = ceil_div(T > 0 ? T : 1, BM) * BM;
  if (rows > t_pad) rows = t_pad;
  L.chunk_rows = rows;
  L.ldg = ceil_div(V, BN) * BN;
  L.g = 0;
  L.total = align_up((size_t)rows * (size_t)L.ldg * 2, 256);
  return L;
}

cudaError_t launch_bwd_bf16(const void* H, const void* W, const int32_t* y, const float* lse,
                            const float* coef, float grad_loss, int64_t T, int32_t d, int32_t V,
                            void* dH, int32_t dH_dtype, float* dW, int accumulate,
                            char* ws, const BwdWs& L, int32_t* d_status, cudaStream_t st) {
  __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(ws + L.g);
  if (T == 0) {
    if (!accumulate) return cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)V * d, st);
    return cudaSuccess;
  }
  CUtensorMap mH_k, mW_k, mW_mn, mH_mn;
  if (!make_map(&mH_k, H, d, T, d, BM) || !make_map(&mW_k, W, d, V, d, BN) ||
      !make_map(&mW_mn, W, d, V, d, 64) || !make_map(&mH_mn, H, d, T, d, 64))
    return cudaErrorInvalidValue;
  const int n_tiles_v = (int)ceil_div(V, BN);
  const int n_tiles_d = (int)ceil_div(d, BN);
  cudaError_t e;
  int chunk = 0;
  for (int64_t t0 = 0; t0 < T; t0 += L.chunk_rows, ++chunk) {
    const int64_t rows = (T - t0) < L.chunk_rows ? (T - t0) : L.chunk_rows;
    const int m_tiles = (int)ceil_div(rows, BM);
    CUtensorMap mG_k, mG_mn;
    if (!make_map(&mG_k, G, V, rows, L.ldg, BM) || !make_map(&mG_mn, G, V, rows, L.ldg, 64))
      return cudaErrorInvalidValue;
    // 1) logits of the chunk, rewritten in place as g (bf16)
    {
      GemmParams p{};
      p.m_tiles = m_tiles;
      p.n_tiles = n_tiles_v;
      int nsplit = pick_fwd_split(m_tiles, n_tiles_v);
      p.per_split = (int)ceil_div(n_tiles_v, nsplit);
      p.nsplit = (int)ceil_div(n_tiles_v, p.per_split);
      p.k_blocks = (int)ceil_div(d, BK);
      p.a_row0 = (int)t0;
      p.rows_valid = T;
      p.cols_valid = V;
      p.out_row0 = t0;
      p.y = y; p.lse = lse; p.coef = coef; p.grad_loss = grad_loss;
      p.T = T;
      p.G = G; p.ldg = L.ldg;
      p.d_status = d_status;
      if ((e = launch_gemm<MODE_G>(mH_k, mW_k, p, st)) != cudaSuccess) return e;
    }
    // 2) dH rows of the chunk = G W
    {
      GemmParams p{};
      p.m_tiles = m_tiles;
      p.n_tiles = n_tiles_d;
      p.nsplit = n_tiles_d;
      p.per_split = 1;
      p.k_blocks = (int)ceil_div(V, BK);
      p.a_row0 = 0;
      p.b_k0 = 0;
      p.rows_valid = T;
      p.cols_valid = d;
      p.out_row0 = t0;
      p.out = dH; p.out_bf16 = (dH_dtype == SPO_DTYPE_BF16); p.ldo = d; p.accumulate = 0;
      p.d_status = d_status;
      if ((e = launch_gemm<MODE_DH>(mG_k, mW_mn, p, st)) != cudaSuccess) return e;
    }
    // 3) dW (+)= G^T H_chunk
    {
      GemmParams p{};
      p.m_tiles = (int)ceil_div(V, BM);
      p.n_tiles = n_tiles_d;
      p.nsplit = n_tiles_d;
      p.per_split = 1;
      p.k_blocks = (int)ceil_div(rows, BK);
      p.a_row0 = 0;
      p.b_k0 = (int)t0;
      p.rows_valid = V;
      p.cols_valid = d;
      p.out_row0 = 0;
      p.out = dW; p.out_bf16 = 0; p.ldo = d; p.accumulate = (accumulate || chunk > 0) ? 1 : 0;
      p.d_status = d_status;
      if ((e = launch_gemm<MODE_DW>(mG_mn, mH_mn, p, st)) != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

}  // namespace spo
