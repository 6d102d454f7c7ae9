// Several sequences through ONE pass over the weights (the batched, KV-heavy form of the verify
// step: the method's premise is that a target call is bound by streaming the parameters, Sec. 1 and
// Sec. 4 "Metrics", so B sequences should share that stream).  The rows of all sequences --
// B x (gamma + 1) for a verify step, B x 2 for a draft step -- go through each projection as one
// dense GEMM on the tcgen05 tensor cores (spd_prefill.cuh); attention, rotary embedding, cache
// append, the rejection rule and the commit stay per sequence: every sequence has its own cache,
// its own length and its own accepted count (Sec. 2.1's rule is stated per sequence).
#pragma once
#include "spd_kernel.cuh"

namespace spd {

struct BatchSeq {
  DevState* st;
  int pos_base_t, pos_base_d;   // rows in front of the text in the target's / draft's cache
};

constexpr int BATCH_ROWS_MAX = 128;   // one 128-row tile of the tensor-core GEMM

// Row (b, m) of a batched launch.  Verify: m = 0 the pending token, m >= 1 draft token m-1, cache row
// and rotary position origin_b + m.  Draft step j: the two rows [token before, token to extend] at
// origin_b + j - 1 + m (as in the single-sequence step).  Writes the embedding rows, each row's
// absolute cache row, and each sequence's origin.  An id outside [0, V) is read as 0 and reported.
__global__ void batch_embed_kernel(const BatchSeq* seqs, int B, int M, int draft, int j, const float* table, int d,
                                   int V, float* X, int* rowslot, int* origins, int* err) {
  const int r = blockIdx.x, b = r / M, m = r - b * M;
  const DevState* st = seqs[b].st;
  const int origin = (draft ? seqs[b].pos_base_d : seqs[b].pos_base_t) + st->n_text;
  int id, slot;
  if (draft) {
    const int t = j - 1 + m;
    id = t < 0 ? st->prev : (t == 0 ? st->pending : st->d_ids[t - 1]);
    slot = origin + t;
  } else {
    id = m == 0 ? st->pending : st->d_ids[m - 1];
    slot = origin + m;
  }
  if ((unsigned)id >= (unsigned)V) {
    if (threadIdx.x == 0) atomicCAS(err, DEV_OK, DEV_BAD_TOKEN);
    id = 0;
  }
  if (threadIdx.x == 0) { rowslot[r] = slot; if (m == 0) origins[b] = origin; }
  const float4* src = reinterpret_cast<const float4*>(table + (size_t)id * d);
  float4* dst = reinterpret_cast<float4*>(X + (size_t)r * d);
  for (int i = threadIdx.x; i < (d >> 2); i += blockDim.x) dst[i] = src[i];
}

// qkv fp32 [R][3d] (natural row order) -> rotary embedding on q and k at each row's own position
// (pairs (i, i + dh/2)); q goes to its sequence's query rows [M][d] (fp32), k and v are appended
// to its sequence's cache at the row's cache row.
// `qkv` may be the sum of `slices` partial products [slices][R][3d] (K slices of the projection, added in
// slice order as tc_reduce_kernel does).
__global__ void batch_rope_append_kernel(const float* qkv, int slices, int R, int M, int d, int dh, const int* rowslot,
                                         const float* cs, const float* sn, const ModelDev* mds, int layer) {
  const size_t sstride = (size_t)R * 3 * d;
  auto at = [&](const float* p) {
    float v = 0.f;
    for (int s = 0; s < slices; ++s) v += p[(size_t)s * sstride];
    return v;
  };
  const int half = dh >> 1, pairs = d >> 1;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)R * pairs;
       i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / pairs), p = (int)(i - (size_t)r * pairs);
    const int b = r / M, m = r - b * M;
    const int h = p / half, jj = p - h * half;
    const int c0 = h * dh + jj, c1 = c0 + half;
    const int pos = rowslot[r];
    const float* row = qkv + (size_t)r * 3 * d;
    const float c = cs[(size_t)pos * half + jj], s = sn[(size_t)pos * half + jj];
    const float qa = at(row + c0), qb = at(row + c1), ka = at(row + d + c0), kb = at(row + d + c1);
    const ModelDev& md = mds[b];
    float* q = md.qbuf + (size_t)m * d;
    q[c0] = qa * c - qb * s;
    q[c1] = qb * c + qa * s;
    const size_t crow = (((size_t)layer * md.H + h) * md.max_seq + pos) * dh;   // cache: [L][H][max_seq][dh]
    __nv_bfloat16* kc = static_cast<__nv_bfloat16*>(md.kcache) + crow;
    __nv_bfloat16* vc = static_cast<__nv_bfloat16*>(md.vcache) + crow;
    kc[jj] = __float2bfloat16_rn(ka * c - kb * s);
    kc[jj + half] = __float2bfloat16_rn(kb * c + ka * s);
    vc[jj] = __float2bfloat16_rn(at(row + 2 * d + c0));
    vc[jj + half] = __float2bfloat16_rn(at(row + 2 * d + c1));
  }
}

// Attention of every sequence's M rows over its own cache.  Work unit = (sequence, head, KV split),
// the single-sequence unit of attn_phase_mma (partial results of a head merged by the CTA that
// finishes its last split); the units of ALL sequences form one list that a grid of persistent CTAs
// walks with stride gridDim.x, so a CTA's next unit usually belongs to another sequence and no CTA
// waits for another.  `chain0`: block-row offset of row 0 (verify: 0; draft step j: j - 1); row m
// attends the rows from the origin up to its own.
// `max_split`: KV splits per head at most -- with B sequences there are enough (sequence, head) pairs
// to fill the grid, so heads are cut no further than needed (fewer partial results to merge).
// o_hi / o_lo: every sequence's output rows as one matrix [B * M][d] split into bf16 hi + lo (the
// operand of the output projection).
template <int M>
__global__ void __launch_bounds__(CONSUMER_THREADS, 2) batch_attn_kernel(const ModelDev* mds, const int* origins, int B,
                                                                      int layer, int chain0, int xbytes, int max_split,
                                                                      __nv_bfloat16* o_hi, __nv_bfloat16* o_lo) {
  extern __shared__ __align__(1024) char bsm[];
  Ctrl* ctl = reinterpret_cast<Ctrl*>(bsm);
  char* xs = bsm + CTRL_BYTES;
  if (threadIdx.x < M) {
    const int top = chain0 + (int)threadIdx.x;          // highest block row this row attends (-1: none)
    ctl->sees[threadIdx.x] = top < 0 ? 0u : ((2u << top) - 1u);
  }
  __syncthreads();
  const int umax = mds[0].H * max_split;                // most units a sequence can have
  for (int g = blockIdx.x; g < B * umax; g += gridDim.x) {
    const int b = g / umax, u = g - b * umax;
    ModelDev md = mds[b];
    md.nsplit = max_split;
    const int units = md.H * eff_nsplit(md, origins[b] + chain0 + M);
    if (u >= units) continue;
    // one unit: the phase's own loop runs once for "CTA u of a grid of `units`"
    const size_t row0 = (size_t)b * M * md.d;
    attn_phase_mma<M, true>(md, layer, origins[b], chain0 + M, u, units, xs, xbytes, ctl, o_hi + row0, o_lo + row0);
    named_sync(1, CONSUMER_THREADS);
  }
}

// softmax(logits / T) of each row (one CTA per row), the same arithmetic per element as the
// single-sequence path: exp(l / T - max) / sum, each step one IEEE operation.
__global__ void __launch_bounds__(SAMPLE_THREADS) batch_softmax_kernel(const float* logits, int V, float temperature,
                                                                       float* probs) {
  __shared__ float red[8];
  const float* row = logits + (size_t)blockIdx.x * V;
  float* out = probs + (size_t)blockIdx.x * V;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float mx = -INFINITY;
  for (int k = threadIdx.x; k < V; k += SAMPLE_THREADS) mx = fmaxf(mx, __fdiv_rn(row[k], temperature));
#pragma unroll
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  mx = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
  __syncthreads();
  float sum = 0.f;
  for (int k = threadIdx.x; k < V; k += SAMPLE_THREADS) sum += expf(__fsub_rn(__fdiv_rn(row[k], temperature), mx));
#pragma unroll
  for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) red[warp] = sum;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  for (int k = threadIdx.x; k < V; k += SAMPLE_THREADS)
    out[k] = __fdiv_rn(expf(__fsub_rn(__fdiv_rn(row[k], temperature), mx)), tot);
}

// Draft step j of every sequence (one CTA each): x_j drawn from the sequence's row of q_j (rows
// [B][2][V], the second row of a sequence is the token being extended), or its arg-max of the
// logits when greedy; q_j is kept as row j of the sequence's draft distributions [B][gamma][V].
__global__ void __launch_bounds__(SAMPLE_THREADS) batch_draft_sample_kernel(const BatchSeq* seqs, const float* rows,
                                                                            int V, int gamma, int j, int greedy,
                                                                            const float* u, float* q_all) {
  __shared__ SampleScratch sc;
  const int b = blockIdx.x;
  const float* row = rows + ((size_t)b * 2 + 1) * V;
  int tok;
  if (greedy) {
    tok = block_argmax([&](int k) { return row[k]; }, V, &sc);
  } else {
    tok = block_sample([&](int k) { return row[k]; }, V, u[(size_t)b * gamma + j], &sc);
    float* q = q_all + ((size_t)b * gamma + j) * V;
    for (int k = threadIdx.x; k < V; k += SAMPLE_THREADS) q[k] = row[k];
  }
  if (threadIdx.x == 0) seqs[b].st->d_ids[j] = tok;
}

// The rejection rule and the commit, one CTA per sequence (Sec. 2.1): rows [B][gamma+1][V] are the
// target's probability rows (logit rows when greedy: only their arg-max is used), q_all
// [B][gamma][V] the draft's.  Each sequence advances by its own accepted count.
__global__ void __launch_bounds__(SAMPLE_THREADS) batch_verify_kernel(const BatchSeq* seqs, const float* rows,
                                                                      const float* q_all, const float* u, int gamma,
                                                                      int V, int greedy, int* n_acc, int* next) {
  __shared__ SampleScratch sc;
  __shared__ int s_ids[MAX_M];
  const int b = blockIdx.x;
  DevState* st = seqs[b].st;
  if (threadIdx.x < gamma) {
    const int x = st->d_ids[threadIdx.x];
    s_ids[threadIdx.x] = (unsigned)x < (unsigned)V ? x : 0;   // the embedding kernel has flagged it
  }
  named_sync(1, SAMPLE_THREADS);
  int r, tok;
  reject_rule_block(rows + (size_t)b * (gamma + 1) * V, q_all + (size_t)b * gamma * V, s_ids,
                    u ? u + (size_t)b * (gamma + 1) : nullptr, gamma, V, greedy, &sc, r, tok);
  if (threadIdx.x == 0) {
    st->n_acc = r;
    st->next = tok;
    st->n_text += r + 1;
    st->prev = r >= 1 ? s_ids[r - 1] : st->pending;
    st->pending = tok;
    st->block += 1;
    if (n_acc) n_acc[b] = r;
    if (next) next[b] = tok;
  }
}

}  // namespace spd
