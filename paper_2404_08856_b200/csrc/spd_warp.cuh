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
// Bin totals are kept as two 32-bit sums (low 16 bits, the rest), which 32-bit shared-memory
// atomics add exactly.
#pragma once
#include "spd_sample.cuh"

namespace spd {

constexpr int WARP_THREADS = 256;

struct TruncScratch {
  unsigned int hlo[256], hhi[256];   // per-bin totals as sum(v & 0xffff) and sum(v >> 16): 32-bit atomics, exact 64-bit result
  unsigned long long suf[256];       // suffix totals of the bins (bins above b)
  unsigned long long red[8];
  unsigned long long wred[8];
  unsigned int seg[WARP_THREADS];
  unsigned long long rem;   // count or mass still to be taken at the current level
  unsigned int chosen;
  unsigned int top;         // largest top byte present
  int found;
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

__device__ __forceinline__ unsigned long long bin_total(const TruncScratch* sc, int b) {
  return ((unsigned long long)sc->hhi[b] << 16) + sc->hlo[b];
}
__device__ __forceinline__ void bin_add(TruncScratch* sc, unsigned b, unsigned long long v) {
  atomicAdd(&sc->hlo[b], (unsigned)(v & 0xffffull));
  atomicAdd(&sc->hhi[b], (unsigned)(v >> 16));
}

// Thread b owns bin b.  Finds the bin in which the running total from the top bin downwards
// crosses sc->rem, stores it in sc->chosen and reduces sc->rem to what is still needed inside it.
// Returns false (all threads) if the bins together do not reach rem.
__device__ bool pick_bin(TruncScratch* sc) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned long long h = bin_total(sc, tid);
  // totals of the bins above tid: suffix scan inside the warp (towards higher lanes), then across warps
  unsigned long long incl = h;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += t;
  }
  if (lane == 0) sc->wred[warp] = incl;
  if (tid == 0) sc->found = 0;
  __syncthreads();
  unsigned long long above = incl - h;
  for (int w = warp + 1; w < WARP_THREADS / 32; ++w) above += sc->wred[w];
  const unsigned long long rem = sc->rem;
  __syncthreads();
  if (h > 0 && above < rem && rem <= above + h) { sc->chosen = (unsigned)tid; sc->rem = rem - above; sc->found = 1; }
  __syncthreads();
  return sc->found != 0;
}

// Keeps the first tokens of the order until `target` is reached (MASS: their mass, else their
// number); the others get the marker -1.  Rows entries < 0 are already excluded.  Requires
// 1 <= target <= total count / mass of the entries still kept.
// The cut is found digit by digit (8 bits at a time) over the fp32 bit patterns.  Probabilities
// share a handful of exponents, so the first digit would send every thread's atomics to a few
// bins: it is counted in registers instead, over the 16 values below the largest top byte present
// (everything lower goes to one "rest" total); only if the cut falls into the rest is the first
// digit redone with atomics over the lower values.
template <bool MASS>
__device__ void truncate_pass(float* row, int V, unsigned long long target, TruncScratch* sc) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned int prefix = 0;
  if (tid == 0) { sc->rem = target; sc->top = 0; }
  sc->hlo[tid] = 0; sc->hhi[tid] = 0;
  __syncthreads();
  {  // largest top byte among the kept entries
    unsigned int mb = 0;
    for (int i = tid; i < V; i += WARP_THREADS) {
      const float w = row[i];
      if (w >= 0.0f) mb = max(mb, __float_as_uint(w) >> 24);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    if (lane == 0) atomicMax(&sc->top, mb);
  }
  __syncthreads();
  const unsigned int top = sc->top;
  {  // first digit: window [top-15, top] in registers, the rest lumped
    constexpr int WIN = 16;
    unsigned long long acc[WIN], rest = 0;
#pragma unroll
    for (int k = 0; k < WIN; ++k) acc[k] = 0;
    for (int i = tid; i < V; i += WARP_THREADS) {
      const float w = row[i];
      if (w < 0.0f) continue;
      const unsigned int d = top - (__float_as_uint(w) >> 24);
      const unsigned long long v = MASS ? to_fixed(w) : 1ull;
      if (d >= WIN) rest += v;
#pragma unroll
      for (int k = 0; k < WIN; ++k) acc[k] += (d == (unsigned)k) ? v : 0ull;
    }
#pragma unroll
    for (int k = 0; k < WIN; ++k) {
      unsigned long long v = acc[k];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && v && top >= (unsigned)k) bin_add(sc, top - k, v);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) rest += __shfl_xor_sync(0xffffffffu, rest, o);
    (void)warp;
    __syncthreads();
    if (!pick_bin(sc)) {
      // the cut lies below the window: take the window's total off and histogram the lower top bytes
      unsigned long long win = 0;
      if (tid == 0) {
        for (int k = 0; k < WIN && (int)top - k >= 0; ++k) win += bin_total(sc, top - k);
        sc->rem -= win;
      }
      __syncthreads();
      sc->hlo[tid] = 0; sc->hhi[tid] = 0;
      __syncthreads();
      for (int i = tid; i < V; i += WARP_THREADS) {
        const float w = row[i];
        if (w < 0.0f) continue;
        const unsigned int byte = __float_as_uint(w) >> 24;
        if (top - byte >= (unsigned)WIN) bin_add(sc, byte, MASS ? to_fixed(w) : 1ull);
      }
      __syncthreads();
      pick_bin(sc);
    }
    prefix = sc->chosen << 24;
  }
  for (int level = 1; level < 4; ++level) {
    const int shift = 24 - 8 * level;
    __syncthreads();
    sc->hlo[tid] = 0; sc->hhi[tid] = 0;
    __syncthreads();
    for (int i = tid; i < V; i += WARP_THREADS) {
      const float w = row[i];
      if (w < 0.0f) continue;
      const unsigned int bits = __float_as_uint(w);
      if ((bits >> (shift + 8)) == (prefix >> (shift + 8))) bin_add(sc, (bits >> shift) & 255u, MASS ? to_fixed(w) : 1ull);
    }
    __syncthreads();
    pick_bin(sc);
    prefix |= sc->chosen << shift;
  }
  __syncthreads();
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
