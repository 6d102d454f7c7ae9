// Tree-based verification (the paper's Sec. 5 names tree-based decoding as the next step and cites
// token-tree systems without defining a rule).  The reading built here is the multi-candidate
// rejection rule of those systems, which keeps the guarantee of Sec. 2.1 (emitted tokens follow the
// target's distribution) when the candidates at a node are drawn independently from the draft's
// distribution at that node.  Letters: p = target, q = draft.
//
// Block rows: 0 = root (the pending token), 1..n = draft nodes, parents first.  P[i] = target's
// distribution after row i, Q[i] = draft's distribution at row i (its children were drawn from it).
// Starting at node = root with cur = P[root]: the children of node are tried in row order; child c
// is accepted iff u[c-1] < min(1, cur[x_c] / Q[node][x_c]); on acceptance node = c, cur = P[c]; on
// rejection cur <- max(0, cur - Q[node]) / its sum and the next child is tried; when no child is
// left the next token is drawn from cur with u[n].  After the LAST child of a node the draw takes
// the un-normalised residual (the integer inverse CDF normalises by its own total), which makes a
// chain-shaped tree identical to the plain rule bit for bit.  Between siblings the residual is
// divided by S = float(Z) * 2^-32 with Z the integer mass of the weights (order independent).
// Greedy: a child is accepted iff its token is the arg-max of P[node]; otherwise that arg-max is
// emitted.  The forward kernel has appended every node's K/V at cache row origin + node; after the
// rule the rows of the accepted nodes move up to origin + depth (tree_gather / tree_scatter).
#pragma once
#include "spd_kernel.cuh"

namespace spd {

// ---- draft side: the children of the rows a draft launch has just computed
// Row k of this launch (k < a.stat_n) is block row node = a.geo.slot[a.stat_r0 + k].  Sampling:
// its probability row prow[k] is stored as Q[node] and every child c is drawn from it with u[c-1]
// (independent draws, repeats allowed).  Greedy: the children are the most probable tokens of the
// row, in order, lower index first among equal logits.
__global__ void __launch_bounds__(SAMPLE_THREADS) tree_draw_kernel(const __grid_constant__ StepArgs a,
                                                                   const TreeShape shape, const float* prow) {
  __shared__ SampleScratch sc;
  __shared__ int taken[MAX_M];
  DevState* st = a.st;
  const int V = a.md.V;
  const float* u = step_uniforms(a, st);
  for (int k = 0; k < a.stat_n; ++k) {
    const int node = a.geo.slot[a.stat_r0 + k];
    const float* lrow = a.logits + (size_t)(a.stat_r0 + k) * V;
    const float* row = prow + (size_t)k * V;
    if (!a.greedy) {
      float* qrow = a.q_out + (size_t)node * V;
      for (int i = threadIdx.x; i < V; i += SAMPLE_THREADS) stcg(qrow + i, ldcg(row + i));
    }
    int n_taken = 0;
    for (int c = 1; c <= shape.n; ++c) {
      if (shape.parent[c] != node) continue;
      int tok;
      if (a.greedy) {
        const int nt = n_taken;
        tok = block_argmax([&](int i) {
          bool used = false;
          for (int t = 0; t < nt; ++t) used |= taken[t] == i;
          return used ? -INFINITY : ldcg(lrow + i);
        }, V, &sc);
        if (threadIdx.x == 0) taken[n_taken] = tok;
        ++n_taken;
        named_sync(1, SAMPLE_THREADS);
      } else {
        tok = block_sample([&](int i) { return ldcg(row + i); }, V, u[c - 1], &sc);
      }
      if (threadIdx.x == 0) st->d_ids[c - 1] = tok;
    }
  }
  if (threadIdx.x == 0) st->t_draft1 = globaltimer();
}

// ---- target side: the rule on the rows of one verify launch, then the commit
// prow [n+1][V] target probability rows (unused when greedy: the arg-max of each row comes from the
// row statistics), q_in [n+1][V] draft rows, cur [V] scratch for a renormalised residual.
__global__ void __launch_bounds__(SAMPLE_THREADS) tree_verify_kernel(const __grid_constant__ StepArgs a,
                                                                     const TreeShape shape, const float* prow,
                                                                     float* cur_buf) {
  __shared__ SampleShared sh;
  __shared__ int s_ids[MAX_M], s_path_ids[MAX_M], s_path[MAX_M];
  DevState* st = a.st;
  const int V = a.md.V, n = shape.n, tid = threadIdx.x;
  const float* u = step_uniforms(a, st);
  if (tid < n) {
    const int x = st->d_ids[tid];
    s_ids[tid] = (unsigned)x < (unsigned)V ? x : 0;   // the forward kernel has flagged it
  }
  if (a.greedy) merge_stats(a.md.stat_part, a.fwd_grid, n + 1, nullptr, sh.rowmax, sh.rowsum, sh.arg);
  named_sync(1, SAMPLE_THREADS);
  int node = 0, plen = 0, tok = 0;
  while (true) {
    const float* cur = prow + (size_t)node * V;        // P[node]; becomes cur_buf after a rejection
    const float* qrow = a.q_in + (size_t)node * V;
    int took = -1, last_child = -1;
    for (int c = 1; c <= n; ++c)
      if (shape.parent[c] == node) last_child = c;
    bool residual = false;                              // the draw below uses max(0, cur - q)
    for (int c = 1; c <= n && took < 0; ++c) {
      if (shape.parent[c] != node) continue;
      const int x = s_ids[c - 1];
      if (a.greedy) {
        if (sh.arg[node] == x) took = c;
        continue;
      }
      if (accept_test(u[c - 1], ldcg(cur + x), ldcg(qrow + x))) { took = c; break; }
      if (c != last_child) {
        // cur <- max(0, cur - q) / sum, the sum taken over integer masses
        unsigned long long z = 0;
        for (int i = tid; i < V; i += SAMPLE_THREADS) z += to_fixed(fmaxf(0.0f, __fsub_rn(ldcg(cur + i), ldcg(qrow + i))));
#pragma unroll
        for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        named_sync(1, SAMPLE_THREADS);
        if ((tid & 31) == 0) sh.sc.wsum[tid >> 5] = z;
        named_sync(1, SAMPLE_THREADS);
        unsigned long long Z = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) Z += sh.sc.wsum[w];
        const float S = __fmul_rn(__ull2float_rn(Z), 2.3283064365386963e-10f);
        for (int i = tid; i < V; i += SAMPLE_THREADS) {
          const float w = fmaxf(0.0f, __fsub_rn(ldcg(cur + i), ldcg(qrow + i)));
          stcg(cur_buf + i, Z ? __fdiv_rn(w, S) : w);
        }
        named_sync(1, SAMPLE_THREADS);
        cur = cur_buf;
      } else {
        residual = true;
      }
    }
    if (took < 0) {
      if (a.greedy) tok = sh.arg[node];
      else if (residual)
        tok = block_sample([&](int i) { return fmaxf(0.0f, __fsub_rn(ldcg(cur + i), ldcg(qrow + i))); }, V, u[n], &sh.sc);
      else
        tok = block_sample([&](int i) { return ldcg(cur + i); }, V, u[n], &sh.sc);
      break;
    }
    if (tid == 0) { s_path[plen] = took; s_path_ids[plen] = s_ids[took - 1]; }
    ++plen;
    node = took;
    named_sync(1, SAMPLE_THREADS);
  }
  named_sync(1, SAMPLE_THREADS);
  if (tid == 0) {
    for (int j = 0; j < plen; ++j) st->path[j] = s_path[j];
    commit_step(a, st, plen, tok, s_path_ids, st->pending);
    st->t_verify1 = globaltimer();
  }
}

// ---- K/V compaction after a tree block: the accepted node at depth j sits in cache row
// origin + path[j-1] and belongs at origin + j.  Rows are first gathered into a staging buffer
// and then scattered, because one accepted node's destination may be another's source.
// grid = (MAX_M - 1, n_layers, 2 {K, V}); `max_depth` caps the moved depths (the draft was never
// fed the deepest level).  commit_step has already advanced n_text by n_acc + 1.
__global__ void tree_gather_kernel(const DevState* st, const ModelDev md, int pos_base, int esz, int max_depth,
                                   char* staging, int scatter) {
  const int j = blockIdx.x + 1, l = blockIdx.y, kv = blockIdx.z;
  const int a = st->n_acc;
  if (j > a || j > max_depth) return;
  const int node = st->path[j - 1];
  if (node == j) return;                                // already in place
  const int origin = pos_base + st->n_text - (a + 1);
  const size_t rowb = (size_t)md.d * esz, headb = (size_t)md.dh * esz;      // a node's row = H pieces of dh
  char* cache = static_cast<char*>(kv ? md.vcache : md.kcache) + (size_t)l * md.max_seq * rowb;   // [H][max_seq][dh]
  char* stg = staging + (((size_t)kv * md.L + l) * MAX_M + j) * rowb;
  const int per_head = (int)(headb >> 4);
  for (int i = threadIdx.x; i < (int)(rowb >> 4); i += blockDim.x) {
    const int h = i / per_head, c = i - h * per_head;
    uint4* in_stage = reinterpret_cast<uint4*>(stg + (size_t)h * headb) + c;
    if (scatter)
      reinterpret_cast<uint4*>(cache + ((size_t)h * md.max_seq + origin + j) * headb)[c] = *in_stage;
    else
      *in_stage = reinterpret_cast<const uint4*>(cache + ((size_t)h * md.max_seq + origin + node) * headb)[c];
  }
}

}  // namespace spd
