// Top-k / top-p (nucleus) truncation of probability rows ahead of the speculative-sampling rule.
// The paper decodes greedily and names sampling with top-p / top-k as future work (Sec. 4
// "Decoding"); truncating and renormalising BOTH the target's and the draft's rows and applying
// the unchanged rule of Sec. 2.1 to them keeps the method's guarantee for the truncated target
// distribution.
//
// Definitions (exact, so that the result does not depend on the order of any reduction):
//   order  larger probability first, lower index first among equal probabilities;
//   mass   W_i = trunc(w_i * 2^32), summed as integers;
//   top-k  the first k tokens of the order;
//   top-p  among the kept tokens (total mass Z) the shortest prefix of the order whose mass
//          reaches T = ceil(Z * trunc(top_p * 2^24) / 2^24), at least one token;
//   output w_i / S for kept tokens with S = float(kept mass) * 2^-32, 0 for the others.
// One CTA per row: the row sits in shared memory, the cut is found by a 4-level radix descent
// over the fp32 bit patterns (monotone for non-negative values) with a histogram of counts
// (top-k) or masses (top-p) per level, ties at the cut value are resolved in index order.
#pragma once
#include "spd_sample.cuh"

namespace spd {

constexpr int WARP_THREADS = 256;

struct TruncScratch {
  unsigned long long hist[256];
  unsigned long long red[8];
  unsigned int seg[WARP_THREADS];
  unsigned long long rem;   // count or mass still to be taken at the current level
  unsigned int chosen;
};

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, TruncScratch* sc) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sc->red[warp] = v;
  __syncthreads();
  unsigned long long t = 0;
#pragma unroll
  for (int w = 0; w < WARP_THREADS / 32; ++w) t += sc->red[w];
  return t;
}

// Keeps the first tokens of the order until `target` is reached (MASS: their mass, else their
// number); the others get the marker -1.  Rows entries < 0 are already excluded.  Requires
// 1 <= target <= total count / mass of the entries still kept.
template <bool MASS>
__device__ void truncate_pass(float* row, int V, unsigned long long target, TruncScratch* sc) {
  const int tid = threadIdx.x;
  unsigned int prefix = 0;
  if (tid == 0) sc->rem = target;
  for (int level = 0; level < 4; ++level) {
    const int shift = 24 - 8 * level;
    sc->hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < V; i += WARP_THREADS) {
      const float w = row[i];
      if (w < 0.0f) continue;
      const unsigned int bits = __float_as_uint(w);
      if (level == 0 || (bits >> (shift + 8)) == (prefix >> (shift + 8)))
        atomicAdd(&sc->hist[(bits >> shift) & 255u], MASS ? to_fixed(w) : 1ull);
    }
    __syncthreads();
    {  // thread b owns bin b: the cut falls into the bin where the running total from the top crosses rem
      unsigned long long above = 0;
      for (int j = 255; j > tid; --j) above += sc->hist[j];
      const unsigned long long rem = sc->rem, h = sc->hist[tid];
      __syncthreads();
      if (h > 0 && above < rem && rem <= above + h) { sc->chosen = (unsigned)tid; sc->rem = rem - above; }
    }
    __syncthreads();
    prefix |= sc->chosen << shift;
  }
  // prefix = bit pattern of the cut value; rem = count / mass still needed from the entries equal to it
  const float cut = __uint_as_float(prefix);
  unsigned long long need = sc->rem;
  if (MASS) {
    const unsigned long long wc = to_fixed(cut);
    need = wc ? (need + wc - 1) / wc : 0xffffffffull;
  }
  const int L = (V + WARP_THREADS - 1) / WARP_THREADS;
  const int i0 = min(V, tid * L), i1 = min(V, i0 + L);
  unsigned int mine = 0;
  for (int i = i0; i < i1; ++i) mine += (row[i] == cut);
  sc->seg[tid] = mine;
  __syncthreads();
  unsigned long long before = 0;
  for (int j = 0; j < tid; ++j) before += sc->seg[j];
  for (int i = i0; i < i1; ++i) {
    const float w = row[i];
    if (w < cut) row[i] = -1.0f;
    else if (w == cut) { if (before >= need) row[i] = -1.0f; ++before; }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(WARP_THREADS)
truncate_rows_kernel(const float* __restrict__ in, float* __restrict__ out, int V, int top_k, float top_p) {
  extern __shared__ float trunc_row[];
  __shared__ TruncScratch sc;
  const float* src = in + (size_t)blockIdx.x * V;
  float* dst = out + (size_t)blockIdx.x * V;
  for (int i = threadIdx.x; i < V; i += WARP_THREADS) {
    const float w = src[i];
    trunc_row[i] = w > 0.0f ? w : 0.0f;
  }
  __syncthreads();
  if (top_k >= 1 && top_k < V) truncate_pass<false>(trunc_row, V, (unsigned long long)top_k, &sc);
  unsigned long long z = 0;
  for (int i = threadIdx.x; i < V; i += WARP_THREADS) {
    const float w = trunc_row[i];
    if (w >= 0.0f) z += to_fixed(w);
  }
  z = block_sum_u64(z, &sc);
  if (top_p > 0.0f && top_p < 1.0f && z > 0) {
    const unsigned long long p24 = static_cast<unsigned long long>(__fmul_rn(top_p, 16777216.0f));
    unsigned long long T = (z * p24 + 16777215ull) >> 24;
    if (T < 1) T = 1;
    truncate_pass<true>(trunc_row, V, T, &sc);
    z = 0;
    for (int i = threadIdx.x; i < V; i += WARP_THREADS) {
      const float w = trunc_row[i];
      if (w >= 0.0f) z += to_fixed(w);
    }
    z = block_sum_u64(z, &sc);
  }
  const float S = __fmul_rn(__ull2float_rn(z), 2.3283064365386963e-10f);   // * 2^-32, exact
  for (int i = threadIdx.x; i < V; i += WARP_THREADS) {
    const float w = trunc_row[i];
    dst[i] = w < 0.0f ? 0.0f : (z ? __fdiv_rn(w, S) : w);
  }
}

}  // namespace spd
