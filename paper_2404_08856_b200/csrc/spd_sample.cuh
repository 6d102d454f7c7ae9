// Block-cooperative sampling primitives (256 threads = 8 warps, named barrier 1).
//
// Drawing from a weight vector w with a uniform u is an inverse-CDF lookup in integers:
// W_k = trunc(w_k * 2^32), Z = sum W_k, t = floor(Z * floor(u * 2^24) / 2^24), result =
// the smallest k whose inclusive prefix sum exceeds t; Z == 0 falls back to argmax(w)
// (lowest index).  Integer sums make the result independent of the reduction tree.
// The acceptance rule and the residual follow Sec. 2.1 of the paper (p = target,
// q = draft): accept iff u < min(1, p/q); replacement ~ max(0, p - q) / sum.
#pragma once
#include "spd_device.cuh"

namespace spd {

constexpr int SAMPLE_THREADS = 256;

struct SampleScratch {
  unsigned long long wsum[8];
  float amax[8];
  int aidx[8];
  float fval[8];
  int result;
  int flag;
};

__device__ __forceinline__ unsigned long long to_fixed(float w) {
  return static_cast<unsigned long long>(__fmul_rn(w, 4294967296.0f));  // cvt.rzi, exact scale
}

__device__ __forceinline__ unsigned long long threshold(unsigned long long Z, float u) {
  const unsigned long long u24 = static_cast<unsigned long long>(__fmul_rn(u, 16777216.0f));
  const unsigned long long lo = Z * u24, hi = __umul64hi(Z, u24);
  return (hi << 40) | (lo >> 24);
}

// min(1, p/q) with one IEEE division; q == 0 accepts iff p > 0.
__device__ __forceinline__ bool accept_test(float u, float p, float q) {
  float a;
  if (q == 0.0f) a = p > 0.0f ? 1.0f : 0.0f;
  else a = fminf(1.0f, __fdiv_rn(p, q));
  return u < a;
}

// All 256 threads call this; wf(k) -> weight >= 0 of index k, must be a pure function.
template <class WF>
__device__ int block_sample(WF wf, int V, float u, SampleScratch* sc) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int VW = (((V + 7) >> 3) + 31) & ~31;
  const int k0 = warp * VW, k1 = min(V, k0 + VW);
  unsigned long long s = 0;
  float bm = -1.0f;
  int bi = 0x7fffffff;
  for (int k = k0 + lane; k < k1; k += 32) {
    const float w = wf(k);
    s += to_fixed(w);
    if (w > bm) { bm = w; bi = k; }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    const float om = __shfl_xor_sync(0xffffffffu, bm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (om > bm || (om == bm && oi < bi)) { bm = om; bi = oi; }
  }
  if (lane == 0) { sc->wsum[warp] = s; sc->amax[warp] = bm; sc->aidx[warp] = bi; }
  named_sync(1, SAMPLE_THREADS);
  unsigned long long Z = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) Z += sc->wsum[w];
  if (Z == 0) {
    float m = sc->amax[0];
    int idx = sc->aidx[0];
#pragma unroll
    for (int w = 1; w < 8; ++w)
      if (sc->amax[w] > m) { m = sc->amax[w]; idx = sc->aidx[w]; }
    named_sync(1, SAMPLE_THREADS);
    return idx;
  }
  const unsigned long long T = threshold(Z, u);
  unsigned long long base = 0;
  int ww = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    if (T >= base + sc->wsum[w] && w == ww) { base += sc->wsum[w]; ww = w + 1; }
  }
  if (ww > 7) ww = 7;  // cannot happen (T < Z); keeps indices in range
  if (warp == ww) {
    int found = k1 - 1;
    for (int kb = k0; kb < k1; kb += 32) {
      const int k = kb + lane;
      unsigned long long inc = (k < k1) ? to_fixed(wf(k)) : 0ull;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const unsigned long long tot = __shfl_sync(0xffffffffu, inc, 31);
      if (T < base + tot) {
        const unsigned mask = __ballot_sync(0xffffffffu, base + inc > T);
        found = kb + __ffs(mask) - 1;
        break;
      }
      base += tot;
    }
    if (lane == 0) sc->result = found;
  }
  named_sync(1, SAMPLE_THREADS);
  const int r = sc->result;
  named_sync(1, SAMPLE_THREADS);
  return r;
}

// The same draw spread over the grid.  Step 1, every CTA: integer mass and largest weight of its
// contiguous vocabulary slice [cta * VS, (cta + 1) * VS) -> part[cta].  Step 2 (after a grid
// barrier), one CTA: the slice in which the running total crosses the threshold, then the token
// inside it.  Integer sums make the result identical to block_sample's.
template <class WF>
__device__ void slice_mass(WF wf, int V, int cta, int G, unsigned long long* part, SampleScratch* sc) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int VS = (V + G - 1) / G;
  const int k0 = cta * VS, k1 = min(V, k0 + VS);
  unsigned long long s = 0;
  float bm = -1.0f;
  int bi = 0x7fffffff;
  for (int k = k0 + tid; k < k1; k += SAMPLE_THREADS) {
    const float w = wf(k);
    s += to_fixed(w);
    if (w > bm) { bm = w; bi = k; }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    const float om = __shfl_xor_sync(0xffffffffu, bm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (om > bm || (om == bm && oi < bi)) { bm = om; bi = oi; }
  }
  if (lane == 0) { sc->wsum[warp] = s; sc->amax[warp] = bm; sc->aidx[warp] = bi; }
  named_sync(1, SAMPLE_THREADS);
  if (tid == 0) {
    unsigned long long z = 0;
    float m = -1.0f;
    int idx = 0x7fffffff;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      z += sc->wsum[w];
      if (sc->amax[w] > m || (sc->amax[w] == m && sc->aidx[w] < idx)) { m = sc->amax[w]; idx = sc->aidx[w]; }
    }
    __stcg(part + 2 * cta, z);
    __stcg(part + 2 * cta + 1, ((unsigned long long)__float_as_uint(fmaxf(m, 0.0f)) << 32) | (unsigned)idx);
  }
  named_sync(1, SAMPLE_THREADS);
}

// All 256 threads of ONE CTA call this after every CTA's slice_mass is visible (grid barrier).
template <class WF>
__device__ int pick_from_slices(WF wf, int V, int G, const unsigned long long* part, float u, SampleScratch* sc) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int VS = (V + G - 1) / G;
  if (tid < 32) {
    constexpr int CH = 8;                       // up to 256 slices
    unsigned long long v[CH];
    unsigned long long Z = 0;
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      const int c = i * 32 + lane;
      v[i] = c < G ? __ldcg(part + 2 * c) : 0ull;
      Z += v[i];
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
    int found;
    if (Z == 0) {
      // no mass at all (underflow): the largest weight, lowest index on ties
      float bm = -1.0f;
      int bi = 0x7fffffff;
      for (int c = lane; c < G; c += 32) {
        const unsigned long long pk = __ldcg(part + 2 * c + 1);
        const float m = __uint_as_float((unsigned)(pk >> 32));
        const int idx = (int)(unsigned)pk;
        if (idx != 0x7fffffff && (m > bm || (m == bm && idx < bi))) { bm = m; bi = idx; }
      }
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, bm, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (om > bm || (om == bm && oi < bi)) { bm = om; bi = oi; }
      }
      found = bi == 0x7fffffff ? 0 : bi;
    } else {
      const unsigned long long T = threshold(Z, u);
      unsigned long long base = 0;
      int cs = G - 1;
      bool hit = false;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        unsigned long long inc = v[i];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += t;
        }
        const unsigned long long tot = __shfl_sync(0xffffffffu, inc, 31);
        if (!hit && T < base + tot) {
          const unsigned mask = __ballot_sync(0xffffffffu, base + inc > T);
          const int l = __ffs(mask) - 1;
          cs = i * 32 + l;
          base += __shfl_sync(0xffffffffu, inc - v[i], l);
          hit = true;
        }
        if (!hit) base += tot;
      }
      const int k0 = min(V, cs * VS), k1 = min(V, k0 + VS);
      found = k1 - 1;
      for (int kb = k0; kb < k1; kb += 32) {
        const int k = kb + lane;
        unsigned long long inc = (k < k1) ? to_fixed(wf(k)) : 0ull;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += t;
        }
        const unsigned long long tot = __shfl_sync(0xffffffffu, inc, 31);
        if (T < base + tot) {
          const unsigned mask = __ballot_sync(0xffffffffu, base + inc > T);
          found = kb + __ffs(mask) - 1;
          break;
        }
        base += tot;
      }
    }
    if (lane == 0) sc->result = found;
  }
  named_sync(1, SAMPLE_THREADS);
  const int r = sc->result;
  named_sync(1, SAMPLE_THREADS);
  return r;
}

// argmax with lowest index on ties over f(k), k < V; all 256 threads call.
template <class F>
__device__ int block_argmax(F f, int V, SampleScratch* sc) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float bm = -INFINITY;
  int bi = 0x7fffffff;
  for (int k = tid; k < V; k += SAMPLE_THREADS) {
    const float w = f(k);
    if (w > bm || bi == 0x7fffffff) { bm = w; bi = k; }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, bm, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (oi != 0x7fffffff && (bi == 0x7fffffff || om > bm || (om == bm && oi < bi))) { bm = om; bi = oi; }
  }
  if (lane == 0) { sc->amax[warp] = bm; sc->aidx[warp] = bi; }
  named_sync(1, SAMPLE_THREADS);
  float m = sc->amax[0];
  int idx = sc->aidx[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) {
    const int oi = sc->aidx[w];
    if (oi != 0x7fffffff && (idx == 0x7fffffff || sc->amax[w] > m || (sc->amax[w] == m && oi < idx))) {
      m = sc->amax[w];
      idx = oi;
    }
  }
  named_sync(1, SAMPLE_THREADS);
  return idx;
}

// The rejection rule (Sec. 2.1) on given probability rows, run by one CTA of SAMPLE_THREADS threads:
// pb [gamma+1][V] target rows, qb [gamma][V] draft rows (unused when greedy), idb [gamma] draft ids
// (each already known to lie in [0, V)), ub [gamma+1] uniforms.  Returns the accepted count in r and
// the next token in tok (the same values in every thread).
__device__ void reject_rule_block(const float* pb, const float* qb, const int* idb, const float* ub, int gamma, int V,
                                  int greedy, SampleScratch* sc, int& r, int& tok) {
  r = gamma;
  if (greedy) {
    tok = -1;
    for (int j = 0; j <= gamma; ++j) {
      const float* row = pb + (size_t)j * V;
      tok = block_argmax([&](int k) { return row[k]; }, V, sc);
      if (j < gamma && tok != idb[j]) { r = j; break; }
    }
  } else {
    for (int j = 0; j < gamma; ++j) {
      const int x = idb[j];
      if (!accept_test(ub[j], pb[(size_t)j * V + x], qb[(size_t)j * V + x])) { r = j; break; }
    }
    const float* prow = pb + (size_t)r * V;
    if (r < gamma) {
      const float* qrow = qb + (size_t)r * V;
      tok = block_sample([&](int k) { return fmaxf(0.0f, __fsub_rn(prow[k], qrow[k])); }, V, ub[gamma], sc);
    } else {
      tok = block_sample([&](int k) { return prow[k]; }, V, ub[gamma], sc);
    }
  }
}

// The rejection rule on given probability rows: one block per sequence.
__global__ void __launch_bounds__(SAMPLE_THREADS)
reject_sample_kernel(const float* __restrict__ p, const float* __restrict__ q, const int* __restrict__ ids,
                     const float* __restrict__ u, int gamma, int V, int greedy, int* __restrict__ n_acc,
                     int* __restrict__ next) {
  __shared__ SampleScratch sc;
  const int b = blockIdx.x;
  const float* pb = p + (size_t)b * (gamma + 1) * V;
  const float* qb = q ? q + (size_t)b * gamma * V : nullptr;
  const int* idb = ids + (size_t)b * gamma;
  const float* ub = u ? u + (size_t)b * (gamma + 1) : nullptr;
  // a draft id outside [0, V) cannot index a row: the sequence is reported as n_acc = next = -1
  bool bad = false;
  for (int j = 0; j < gamma; ++j) bad |= (unsigned)idb[j] >= (unsigned)V;
  if (bad) {
    if (threadIdx.x == 0) { n_acc[b] = -1; next[b] = -1; }
    return;
  }
  int r, tok;
  reject_rule_block(pb, qb, idb, ub, gamma, V, greedy, &sc, r, tok);
  if (threadIdx.x == 0) { n_acc[b] = r; next[b] = tok; }
}

}  // namespace spd
