// Prefill (Eq. 1: the target reads [V_1..V_m ; embed(X_1..X_n)] in one pass): dense GEMMs on
// the 5th-generation tensor cores.  C[M,N] = A[M,K] B[N,K]^T with both operands K-major bf16:
// tiles arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a ring of
// shared-memory stages, one thread issues tcgen05.mma (128x128x16 per instruction) with the
// accumulator in tensor memory, and the epilogue reads it back with tcgen05.ld.
//
// Precision: B operands are exact bf16 data (weights, cached K and V).  The A operand
// (activations, probabilities) is fp32 upstream and is fed as TWO bf16 matrices hi + lo
// (x = hi + lo up to 2^-17 |x|): a stage holds the hi tile, the lo tile and ONE B tile of a K
// block, and both products accumulate into the same tensor-memory columns.  Prefill results
// therefore match an fp32 reference to ~1e-5 relative, like the M <= 8 path, at twice the
// tensor work but with every B tile loaded once.
#pragma once
#include <cuda.h>

#include "spd_device.cuh"

namespace spd {

constexpr int TC_BM = 128, TC_BN = 128, TC_BK = 64;
constexpr int TC_STAGES = 2;          // prefill (compute-bound, many tiles): 2 stages, two CTAs per SM
constexpr int TC_STAGES_STREAM = 4;   // few rows against large weights (HBM-bound): 4 stages, one CTA per SM
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2, TC_B_BYTES = TC_BN * TC_BK * 2;
constexpr int TC_STAGE_BYTES = 2 * TC_A_BYTES + TC_B_BYTES;              // A hi | A lo | B = 48 KB
__host__ __device__ constexpr int tc_stage_bytes(int bn) { return 2 * TC_A_BYTES + bn * TC_BK * 2; }          // A hi | A lo | B (bn rows)
__host__ __device__ constexpr int tc_smem_bytes(int stages, int bn = TC_BN) { return stages * tc_stage_bytes(bn) + 1024 + 256; }   // + alignment slack + barriers
constexpr int TC_BN_WIDE = 256;       // streaming form: two weight tiles per activation tile (half the activation re-reads)
constexpr int TC_STAGES_WIDE = 3;     // 3 x 64 KB
constexpr int TC_BN_MID = 160;        // ... or 160 weight rows, where 256-row tiles would leave too many SMs without a CTA
constexpr int TC_STAGES_MID = 4;      // 4 x 52 KB
__host__ __device__ constexpr int tc_tmem_cols(int bn) { return bn <= 128 ? 128 : 256; }   // allocations are powers of two
constexpr int TC_SMEM_BYTES = tc_smem_bytes(TC_STAGES);

// TC_OUT_SWIGLU: the B rows are [gate_0, up_0, gate_1, up_1, ...]; output column i of the hi/lo result
// [M][N/2] is silu(alpha * gate_i) * (alpha * up_i) (the feed-forward block's non-linearity).
enum : int { TC_OUT_F32 = 0, TC_OUT_F32_ADD = 1, TC_OUT_SPLIT = 2, TC_OUT_SWIGLU = 3 };

struct TcArgs {
  int M, N, K;              // A rows, B rows (= output columns), inner dimension
  int split;                // (always 1: A is given as hi and lo maps)
  int mode;                 // TC_OUT_*
  float alpha;              // result scale
  float* out_f32;
  __nv_bfloat16 *out_hi, *out_lo;
  long long ldo, out_batch; // output row stride and per-batch offset, in elements
  int* err;                 // sticky error word (DEV_TIMEOUT_*)
  int ksplit;               // > 1: blockIdx.z is a slice of the K loop (not a batch index); slice s stores its
                            // partial product (alpha applied) at out_f32 + s * M * ldo, summed by tc_reduce_kernel
};

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle: 8-row groups are
// 1024 bytes apart (stride byte offset), leading byte offset 1 (unused for swizzled K-major).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16: D = fp32, A = B = bf16, both K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t tc_idesc(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// GELU in its exact form x * Phi(x), the non-linearity between the two linear layers of the image
// adapter g_theta (Sec. 2.2, Appendix A.1; the paper does not name it, LLaVA's projector uses it).
__device__ __forceinline__ float gelu_exact(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }

// grid = (N tiles, M tiles, batch); 128 threads: thread 0 feeds TMA, thread 32 issues the MMAs,
// all four warps read the accumulator back (warp w owns TMEM lanes 32w..32w+31 = tile rows).
// GELU: the hi/lo output (TC_OUT_SPLIT) is gelu(alpha * accumulator) instead of alpha * accumulator.
template <bool GELU, int STAGES, int BN = TC_BN>
__global__ void __launch_bounds__(128, (STAGES <= 3 && BN == TC_BN) ? 2 : 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
               const __grid_constant__ CUtensorMap map_b, const TcArgs a) {
  constexpr int STAGE_B = tc_stage_bytes(BN);     // bytes of one ring stage
  extern __shared__ uint8_t tc_smem_raw[];
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(stages + STAGES * STAGE_B);
  uint64_t* empty = full + STAGES;
  uint64_t* accum = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  volatile int* err = a.err;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile_n = blockIdx.x, tile_m = blockIdx.y;
  const int z = a.ksplit > 1 ? 0 : (int)blockIdx.z;           // batch index
  const int slice = a.ksplit > 1 ? (int)blockIdx.z : 0;       // slice of the K loop

  if (tid == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(accum, 1);
    mbar_fence_init();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tc_tmem_cols(BN))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int k_all = (a.K + TC_BK - 1) / TC_BK;
  const int k_per = a.ksplit > 1 ? (k_all + a.ksplit - 1) / a.ksplit : k_all;
  const int k_first = slice * k_per;
  const int k_blocks = max(0, min(k_all, k_first + k_per) - k_first);
  const int total = k_blocks;
  if (tid == 0) {
    // ---- TMA producer
    for (int it = 0; it < total; ++it) {
      const int s = it % STAGES;
      const unsigned ph = (it / STAGES) & 1;
      if (!mbar_wait(&empty[s], ph ^ 1u, err, DEV_TIMEOUT_EMPTY)) break;
      mbar_arrive_expect_tx(&full[s], STAGE_B);
      const int kb = k_first + it;
      tma_load_3d(stages + s * STAGE_B, &map_a_hi, kb * TC_BK, tile_m * TC_BM, z, &full[s]);
      tma_load_3d(stages + s * STAGE_B + TC_A_BYTES, &map_a_lo, kb * TC_BK, tile_m * TC_BM, z, &full[s]);
      tma_load_3d(stages + s * STAGE_B + 2 * TC_A_BYTES, &map_b, kb * TC_BK, tile_n * BN, z, &full[s]);
    }
  } else if (tid == 32) {
    // ---- MMA issuer
    bool ok = true;
    for (int it = 0; it < total && ok; ++it) {
      const int s = it % STAGES;
      const unsigned ph = (it / STAGES) & 1;
      ok = mbar_wait(&full[s], ph, err, DEV_TIMEOUT_FULL);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint64_t ah = umma_desc(smem_u32(stages + s * STAGE_B));
      const uint64_t al = umma_desc(smem_u32(stages + s * STAGE_B + TC_A_BYTES));
      const uint64_t bd = umma_desc(smem_u32(stages + s * STAGE_B + 2 * TC_A_BYTES));
#pragma unroll
      for (int k = 0; k < TC_BK / 16; ++k) {   // 32 bytes further along K inside the swizzle atom
        umma_bf16(tmem_base, ah + 2 * k, bd + 2 * k, tc_idesc(BN), (it > 0 || k > 0) ? 1u : 0u);
        umma_bf16(tmem_base, al + 2 * k, bd + 2 * k, tc_idesc(BN), 1u);
      }
      umma_commit(&empty[s]);   // the stage is free once these MMAs have read it
    }
    umma_commit(accum);         // arrives when every MMA above has completed
  }
  __syncwarp();
  // ---- epilogue
  // (a K slice that got no block -- more slices than blocks -- has nothing to wait for and stores zeros)
  const bool done = total == 0 ? true : mbar_wait(accum, 0u, err, DEV_TIMEOUT_FULL);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const int row = tile_m * TC_BM + warp * 32 + lane;
  if (done) {
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 32) {
      uint32_t v[32];
      if (total == 0) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 0u;
      } else {
        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
      }
      const int col0 = tile_n * BN + c0;
      if (row < a.M && col0 < a.N) {
        const long long off = (long long)z * a.out_batch + (long long)slice * a.M * a.ldo + (long long)row * a.ldo + col0;
        const int nv = min(32, a.N - col0);
        // a thread owns 32 consecutive columns of its row: 16-byte stores where the row start
        // and the width allow it (ldo and out_batch multiples of 8, all 32 columns present)
        const bool vec = nv == 32 && (a.ldo & 7) == 0 && (a.out_batch & 7) == 0;
        if (a.mode == TC_OUT_SWIGLU) {
          // this thread's 32 columns are 16 (gate, up) pairs -> 16 output columns from col0 / 2 on
          const long long off2 = (long long)z * a.out_batch + (long long)row * a.ldo + (col0 >> 1);
          const int np = nv >> 1;
          if (np == 16 && (a.ldo & 7) == 0 && (a.out_batch & 7) == 0) {
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              uint32_t hw[4], lw[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float g0 = __uint_as_float(v[2 * (j + 2 * q)]) * a.alpha, u0 = __uint_as_float(v[2 * (j + 2 * q) + 1]) * a.alpha;
                const float g1 = __uint_as_float(v[2 * (j + 2 * q) + 2]) * a.alpha, u1 = __uint_as_float(v[2 * (j + 2 * q) + 3]) * a.alpha;
                const float x0 = (g0 / (1.0f + expf(-g0))) * u0, x1 = (g1 / (1.0f + expf(-g1))) * u1;
                const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
                const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
                hw[q] = *reinterpret_cast<const uint32_t*>(&h);
                lw[q] = *reinterpret_cast<const uint32_t*>(&l);
              }
              *reinterpret_cast<uint4*>(a.out_hi + off2 + j) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
              *reinterpret_cast<uint4*>(a.out_lo + off2 + j) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            }
          } else {
            for (int j = 0; j < np; ++j) {
              const float g0 = __uint_as_float(v[2 * j]) * a.alpha, u0 = __uint_as_float(v[2 * j + 1]) * a.alpha;
              const float x0 = (g0 / (1.0f + expf(-g0))) * u0;
              const __nv_bfloat16 h0 = __float2bfloat16_rn(x0);
              a.out_hi[off2 + j] = h0;
              a.out_lo[off2 + j] = __float2bfloat16_rn(x0 - __bfloat162float(h0));
            }
          }
        } else if (a.mode == TC_OUT_SPLIT) {
          if (vec) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint32_t hw[4], lw[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                float x0 = __uint_as_float(v[j + 2 * q]) * a.alpha, x1 = __uint_as_float(v[j + 2 * q + 1]) * a.alpha;
                if (GELU) { x0 = gelu_exact(x0); x1 = gelu_exact(x1); }
                const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
                const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
                hw[q] = *reinterpret_cast<const uint32_t*>(&h);
                lw[q] = *reinterpret_cast<const uint32_t*>(&l);
              }
              *reinterpret_cast<uint4*>(a.out_hi + off + j) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
              *reinterpret_cast<uint4*>(a.out_lo + off + j) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            }
          } else {
            for (int j = 0; j < nv; j += 2) {
              float x0 = __uint_as_float(v[j]) * a.alpha, x1 = (j + 1 < nv) ? __uint_as_float(v[j + 1]) * a.alpha : 0.f;
              if (GELU) { x0 = gelu_exact(x0); x1 = gelu_exact(x1); }
              const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
              a.out_hi[off + j] = h0;
              a.out_lo[off + j] = __float2bfloat16_rn(x0 - __bfloat162float(h0));
              if (j + 1 < nv) {
                a.out_hi[off + j + 1] = h1;
                a.out_lo[off + j + 1] = __float2bfloat16_rn(x1 - __bfloat162float(h1));
              }
            }
          }
        } else if (a.mode == TC_OUT_F32_ADD) {
          if (vec) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              float4* p4 = reinterpret_cast<float4*>(a.out_f32 + off + j);
              float4 o = *p4;
              o.x += __uint_as_float(v[j]) * a.alpha; o.y += __uint_as_float(v[j + 1]) * a.alpha;
              o.z += __uint_as_float(v[j + 2]) * a.alpha; o.w += __uint_as_float(v[j + 3]) * a.alpha;
              *p4 = o;
            }
          } else {
            for (int j = 0; j < nv; ++j) a.out_f32[off + j] += __uint_as_float(v[j]) * a.alpha;
          }
        } else {
          if (vec) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(a.out_f32 + off + j) =
                  make_float4(__uint_as_float(v[j]) * a.alpha, __uint_as_float(v[j + 1]) * a.alpha,
                              __uint_as_float(v[j + 2]) * a.alpha, __uint_as_float(v[j + 3]) * a.alpha);
          } else {
            for (int j = 0; j < nv; ++j) a.out_f32[off + j] = __uint_as_float(v[j]) * a.alpha;
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    if (!done) for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tc_tmem_cols(BN)) : "memory");
  }
}

// Sum of the K slices of a split GEMM, in slice order (deterministic): out (+)= sum_s part[s].
__global__ void tc_reduce_kernel(const float* part, int slices, size_t n, float* out, int add) {
  for (size_t i = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) * 4; i < n; i += (size_t)gridDim.x * blockDim.x * 4) {
    float4 acc = add ? *reinterpret_cast<const float4*>(out + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < slices; ++s) {
      const float4 p = *reinterpret_cast<const float4*>(part + (size_t)s * n + i);
      acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
    }
    *reinterpret_cast<float4*>(out + i) = acc;
  }
}

// ------------------------------------------------------------------------------ elementwise

__device__ __forceinline__ void store_split(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float x) {
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  hi[i] = h;
  lo[i] = __float2bfloat16_rn(x - __bfloat162float(h));
}

// fp32 [R][K] -> hi/lo bf16 [R][K]
__global__ void split_rows_kernel(const float* x, __nv_bfloat16* hi, __nv_bfloat16* lo, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    store_split(hi, lo, i, x[i]);
}

// RMSNorm of each row (one block per row), output split into hi/lo bf16.
__global__ void __launch_bounds__(256) rms_split_kernel(const float* x, const float* gain, float eps, int d,
                                                        __nv_bfloat16* hi, __nv_bfloat16* lo) {
  __shared__ float red[8];
  const float* row = x + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int k = threadIdx.x; k < d; k += 256) ss += row[k] * row[k];
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float inv = 1.0f / sqrtf(tot / (float)d + eps);
  for (int k = threadIdx.x; k < d; k += 256)
    store_split(hi, lo, (size_t)blockIdx.x * d + k, (row[k] * inv) * gain[k]);
}

// x[row] += sum over the K slices of a projection's partial products (slice order, as
// tc_reduce_kernel adds them), then the RMSNorm of the updated row with `gain`, split into hi/lo
// bf16: one launch instead of the slice sum and the norm.  slices = 0: the residual is already in x.
__global__ void __launch_bounds__(256) resid_rms_split_kernel(float* x, const float* part, int slices, size_t slice_stride,
                                                              const float* gain, float eps, int d, __nv_bfloat16* hi,
                                                              __nv_bfloat16* lo) {
  __shared__ float red[8];
  constexpr int PER = 4096 / 4 / 256;     // float4 per thread: rows of up to 4096 columns stay in registers
  float* row = x + (size_t)blockIdx.x * d;
  const float* prow = part + (size_t)blockIdx.x * d;
  const int d4 = d >> 2;
  float4 v[PER];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int k4 = threadIdx.x + i * 256;
    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k4 < d4) {
      v[i] = reinterpret_cast<const float4*>(row)[k4];
      float4 p[8];   // all slices of this piece travel together, then they are added in slice order
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < slices) p[s] = reinterpret_cast<const float4*>(prow + (size_t)s * slice_stride)[k4];
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < slices) { v[i].x += p[s].x; v[i].y += p[s].y; v[i].z += p[s].z; v[i].w += p[s].w; }
      if (slices > 0) reinterpret_cast<float4*>(row)[k4] = v[i];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float inv = 1.0f / sqrtf(tot / (float)d + eps);
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int k4 = threadIdx.x + i * 256;
    if (k4 < d4) {
      const float4 g = reinterpret_cast<const float4*>(gain)[k4];
      const size_t o = (size_t)blockIdx.x * d + (size_t)k4 * 4;
      store_split(hi, lo, o, (v[i].x * inv) * g.x);
      store_split(hi, lo, o + 1, (v[i].y * inv) * g.y);
      store_split(hi, lo, o + 2, (v[i].z * inv) * g.z);
      store_split(hi, lo, o + 3, (v[i].w * inv) * g.w);
    }
  }
}

// qkv fp32 [R][3d] (natural row order) -> rotary on q and k (pairs (i, i + dh/2)), q split into
// hi/lo [R][d], k and v appended to the cache rows pos0.. (cache of one layer: [H][max_seq][dh]),
// v also transposed to vT [H][dh][rpad].
__global__ void rope_kv_kernel(const float* qkv, int R, int d, int dh, int pos0, const float* cs, const float* sn,
                               __nv_bfloat16* q_hi, __nv_bfloat16* q_lo, __nv_bfloat16* kc, __nv_bfloat16* vc,
                               __nv_bfloat16* vT, int rpad, int max_seq) {
  const int half = dh >> 1, pairs = d >> 1;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)R * pairs;
       i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / pairs), p = (int)(i - (size_t)r * pairs);
    const int h = p / half, j = p - h * half;
    const int c0 = h * dh + j, c1 = c0 + half;
    const float* row = qkv + (size_t)r * 3 * d;
    const float c = cs[(size_t)(pos0 + r) * half + j], s = sn[(size_t)(pos0 + r) * half + j];
    const float qa = row[c0], qb = row[c1], ka = row[d + c0], kb = row[d + c1];
    store_split(q_hi, q_lo, (size_t)r * d + c0, qa * c - qb * s);
    store_split(q_hi, q_lo, (size_t)r * d + c1, qb * c + qa * s);
    const size_t crow = ((size_t)h * max_seq + pos0 + r) * dh;
    kc[crow + j] = __float2bfloat16_rn(ka * c - kb * s);
    kc[crow + j + half] = __float2bfloat16_rn(kb * c + ka * s);
    const __nv_bfloat16 v0 = __float2bfloat16_rn(row[2 * d + c0]), v1 = __float2bfloat16_rn(row[2 * d + c1]);
    vc[crow + j] = v0;
    vc[crow + j + half] = v1;
    vT[((size_t)h * dh + j) * rpad + r] = v0;
    vT[((size_t)h * dh + j + half) * rpad + r] = v1;
  }
}

// Causal softmax of each score row (one block per (head, row)): row r sees columns 0..r.
// Output probabilities split into hi/lo bf16 [H][R][rpad], zero beyond the diagonal.
__global__ void __launch_bounds__(256) softmax_causal_split_kernel(const float* S, int R, int rpad,
                                                                   __nv_bfloat16* hi, __nv_bfloat16* lo) {
  __shared__ float red[8];
  const size_t base = (size_t)blockIdx.x * rpad;
  const int r = blockIdx.x % R, n = r + 1;
  const float* row = S + base;
  float mx = -INFINITY;
  for (int k = threadIdx.x; k < n; k += 256) mx = fmaxf(mx, row[k]);
#pragma unroll
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
  __syncthreads();
  float sum = 0.f;
  for (int k = threadIdx.x; k < n; k += 256) sum += expf(row[k] - mx);
#pragma unroll
  for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  for (int k = threadIdx.x; k < rpad; k += 256)
    store_split(hi, lo, base + k, k < n ? expf(row[k] - mx) / tot : 0.f);
}

// gu fp32 [R][2f] = [gate_0, up_0, gate_1, up_1, ...] -> silu(gate) * up, split into hi/lo [R][f]
// (used where the gate/up projection was cut into K slices and could not apply it in its epilogue)
__global__ void swiglu_split_kernel(const float* gu, int R, int f, __nv_bfloat16* hi, __nv_bfloat16* lo) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)R * f; i += (size_t)gridDim.x * blockDim.x) {
    const size_t r = i / f, c = i - r * f;
    const float g = gu[r * 2 * f + 2 * c], u = gu[r * 2 * f + 2 * c + 1];
    store_split(hi, lo, i, (g / (1.0f + expf(-g))) * u);
  }
}

}  // namespace spd
