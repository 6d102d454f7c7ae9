// The persistent forward kernel: see spd_engine.cuh for the design.
#pragma once
#include "spd_engine.cuh"

namespace spd {

// Commit of a step by one thread: accepted count r, next token tok (Sec. 2.1: x_1..x_r and the
// replacement / bonus token are emitted; the KV length follows the accepted count).
__device__ __forceinline__ void commit_step(const StepArgs& a, DevState* st, int r, int tok, const int* ids, int pending) {
  st->n_acc = r;
  st->next = tok;
  if (a.mode == MODE_ROWS) {           // prefill: the sequence starts here
    st->n_text = a.init_n_text;
    st->prev = a.init_prev;
    st->pending = tok;
    st->block = 0;
    st->n_emitted = 0;
    if (a.out_ids && st->out_cap > 0) { a.out_ids[0] = tok; st->n_emitted = 1; }
  } else {                              // commit x_1..x_r and the next token
    int ne = st->n_emitted;
    if (a.out_ids) {
      for (int j = 0; j < r; ++j)
        if (ne < st->out_cap) a.out_ids[ne++] = ids[j];
      if (ne < st->out_cap) a.out_ids[ne++] = tok;
    }
    st->n_emitted = ne;
    st->n_text += r + 1;
    st->prev = r >= 1 ? ids[r - 1] : pending;
    st->pending = tok;
    st->block += 1;
  }
}

// Greedy decoding (Sec. 4 "Decoding"), run by CTA 0 after the row statistics are merged: a draft
// token is accepted iff it is the argmax of the target's row; the next token is the argmax of the
// first mismatching row, or of row gamma.  Rows r0..r0+gamma of `logits` are p_1..p_{gamma+1}.
// (With sampling the forward kernel stops after the row statistics and the two sampling kernels
// below finish the step.)
template <int M>
__device__ void verify_greedy(const StepArgs& a, const ModelDev& md, DevState* st, Ctrl* ctl, int G, int r0,
                              int gamma, const int* ids /*gamma draft ids*/, int pending) {
  const int tid = threadIdx.x;
  __shared__ int s_arg[MAX_M];
  merge_stats(md.stat_part, G, gamma + 1, ctl, ctl->rowmax, ctl->rowsum, s_arg);
  int r = gamma;
  for (int j = 0; j < gamma; ++j)
    if (s_arg[j] != ids[j]) { r = j; break; }
  if (tid == 0) commit_step(a, st, r, s_arg[r], ids, pending);
  (void)r0;
}

// Greedy draft step j: x_j = argmax of the row whose statistics sit at index 0.
template <int M>
__device__ void draft_greedy(const StepArgs& a, const ModelDev& md, DevState* st, Ctrl* ctl, int G) {
  __shared__ int s_arg[MAX_M];
  merge_stats(md.stat_part, G, 1, ctl, ctl->rowmax, ctl->rowsum, s_arg);
  if (threadIdx.x == 0) st->d_ids[a.j] = s_arg[0];
}

// TRACE: the instantiation that stores phase timestamps (spd_trace).  It is a separate kernel
// because the stamps cost the plain one 1.3 % of the verify step and 3.5 % of a draft step even
// when tracing is off (same-box A/B with the stamps compiled out).
template <int M, typename WT, bool TRACE = false>
__global__ void __launch_bounds__(ENGINE_THREADS, 1) forward_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ __align__(1024) char smem[];
  Ctrl* ctl = reinterpret_cast<Ctrl*>(smem);
  float* red = reinterpret_cast<float*>(smem + CTRL_BYTES + ZERO_BYTES);
  LayerDev* lay_s = reinterpret_cast<LayerDev*>(smem + CTRL_BYTES + ZERO_BYTES + RED_BYTES);
  float* pre_s = reinterpret_cast<float*>(smem + CTRL_BYTES + ZERO_BYTES + RED_BYTES + LAYER_BYTES);
  float* X = reinterpret_cast<float*>(smem + FIXED_SMEM);
  char* stages = smem + FIXED_SMEM + x_bytes(M);
  const uint32_t zero_addr = smem_u32(smem + CTRL_BYTES);
  const ModelDev& md = a.md;
  DevState* st = a.st;
  volatile int* err = &st->err;
  const int tid = threadIdx.x, cta = blockIdx.x, G = gridDim.x;

  if (tid == 0) {
    for (int i = 0; i < a.nstage; ++i) {
      mbar_init(&ctl->full[i], 1);
      mbar_init(&ctl->empty[i], CONSUMER_THREADS / 32);
    }
    mbar_init(&ctl->xbar, 1);
    if (a.cluster_ctas) mbar_init(&ctl->cbar, (unsigned)a.cluster_ctas);
    mbar_fence_init();
  }
  if (tid < ZERO_BYTES / 4) reinterpret_cast<uint32_t*>(smem + CTRL_BYTES)[tid] = 0u;
  // per-layer pointer records: shared memory copy (a dependent global load per projection otherwise)
  const bool lay_in_smem = md.L <= LAYER_SMEM_MAX;
  if (lay_in_smem)
    for (int i = tid; i < md.L * (int)(sizeof(LayerDev) / 8); i += ENGINE_THREADS)
      reinterpret_cast<uint64_t*>(lay_s)[i] = reinterpret_cast<const uint64_t*>(md.layers)[i];
  const LayerDev* layers = lay_in_smem ? lay_s : md.layers;
  __syncthreads();
  // a cluster launch: every member's barrier word must exist before anyone arrives on it
  if (a.cluster_ctas) cluster_sync_all_threads();

  const bool gemm_only = a.mode == MODE_GEMM;
  const bool want_head = gemm_only ? false : (a.mode != MODE_ROWS || a.want_sample);
  const bool head_only = !gemm_only && a.mode == MODE_ROWS && a.skip_layers;
  const int n_layers_run = head_only ? 0 : (gemm_only ? 0 : md.L);
  const int g_first = head_only ? md.L * 4 : 0;
  const int n_gemm = gemm_only ? 1 : n_layers_run * 4 + (want_head ? 1 : 0);

  if (tid >= CONSUMER_THREADS) {
    // ---------------- producer warp: stream every weight tile of this CTA, in order
    Ring ring{0, 0u, a.nstage};
    const uint64_t pol = policy_evict_first();
    if (gemm_only) {
      Gemm g{a.gw, a.gN, a.gK, PRO_PLAIN, EPI_STORE, 0};
      produce_gemm<WT>(g, cta, G, ring, ctl, stages, pol, err);
    } else {
      for (int i = 0; i < n_gemm; ++i) {
        const Gemm g = get_gemm(md, layers, g_first + i);
        produce_gemm<WT>(g, cta, G, ring, ctl, stages, pol, err);
      }
    }
  } else {
    // ---------------- compute warps
    Ring ring{0, 0u, a.nstage};
    unsigned bar_target = 0, xphase = 0, cphase = 0;
    // all CTAs wait for each other: through global memory, or inside the cluster
    auto sync_grid = [&]() {
      if (a.cluster_ctas) cluster_barrier(&ctl->cbar, cphase, (unsigned)G, err);
      else grid_barrier(a.bar, bar_target, G, err);
    };
    if (tid == 0) { ctl->trace = (TRACE && cta == 0) ? a.trace : nullptr; ctl->trace_n = 0; }
    named_sync(1, CONSUMER_THREADS);
    auto stamp = [&](int id = 3) { if constexpr (TRACE) trace_stamp(ctl, id); };
    stamp(0);
    if (cta == 0 && tid == 0) {
      if (a.mode == MODE_VERIFY) st->t_verify0 = globaltimer();
      else if (a.mode == MODE_DRAFT && a.j == 0) st->t_draft0 = globaltimer();
    }
    if (gemm_only) {
      Gemm g{a.gw, a.gN, a.gK, PRO_PLAIN, EPI_STORE, 0};
      EpiArgs e{};
      e.out = a.gy; e.ldo = a.gN;
      const XSrc src{a.gx, (size_t)a.gK, nullptr};
      consume_gemm<M, WT, TRACE>(g, e, src, nullptr, 0.f, nullptr, nullptr, cta, G, ring, ctl, X, xphase, red, pre_s, zero_addr, stages, err);
    } else {
      // origin = sequence position of the pending token; the launch's row table gives each row its
      // token, cache row, rotary position and the block rows it attends
      int origin, pending = 0, nslots;
      int ids[M];
      const bool from_ids = (a.mode != MODE_ROWS) || a.rows == nullptr;
      if (a.mode == MODE_ROWS) {       // a chunk of prompt rows at absolute positions: a chain from rows_pos0
        origin = a.rows_pos0;
        nslots = M;
#pragma unroll
        for (int m = 0; m < M; ++m) ids[m] = a.row_ids ? a.row_ids[m] : 0;
      } else {
        origin = a.pos_base + st->n_text;
        nslots = a.n_slots;
        pending = st->pending;
#pragma unroll
        for (int m = 0; m < M; ++m) {
          const int sr = a.geo.src[m];
          ids[m] = sr == -2 ? st->prev : (sr == -1 ? pending : st->d_ids[sr]);
        }
      }
#pragma unroll
      for (int m = 0; m < M; ++m)
        if (from_ids && (ids[m] < 0 || ids[m] >= md.V)) {
          if (tid == 0) atomicCAS(const_cast<int*>(err), DEV_OK, DEV_BAD_TOKEN);
          ids[m] = 0;
        }
      const int d = md.d, f = md.f;
      // the ids live in shared memory from here on (embedding rows, sampling rule)
      if (tid == 0) {
#pragma unroll
        for (int m = 0; m < M; ++m) {
          ctl->tok[m] = ids[m];
          const bool chain = a.mode == MODE_ROWS;
          ctl->rowslot[m] = origin + (chain ? m : (int)a.geo.slot[m]);
          ctl->rowpos[m] = origin + (chain ? m : (int)a.geo.depth[m]);
          ctl->sees[m] = chain ? ((2u << m) - 1u) : (unsigned)a.geo.sees[m];
        }
      }
      named_sync(1, CONSUMER_THREADS);
      // bf16 models: every residual epilogue leaves x * (gain of the next RMSNorm) in md.xg and
      // per-CTA sums of x^2 in md.ssq, so the norm costs its reader nothing; only the first
      // projection of a launch normalises its rows itself.  fp32 models normalise on load.
      constexpr bool PRE = sizeof(WT) == 2;
      const XSrc src_in = from_ids ? XSrc{md.embed, (size_t)d, ctl->tok} : XSrc{a.rows, (size_t)d, nullptr};
      const XSrc src_x{PRE ? md.xg : md.x, (size_t)d, nullptr};

      // One pass over the projections: index 4l + {0: QKV, 1: O, 2: gate/up, 3: down}, then the LM
      // head.  A single call site keeps one copy of the projection code in the kernel.
      for (int i = 0; i < n_gemm; ++i) {
        const int idx = g_first + i, l = idx >> 2, which = idx & 3;
        const bool head = l >= md.L;
        const Gemm g = get_gemm(md, layers, idx);
        EpiArgs e{};
        XSrc src = src_x;
        const float* norm_w = nullptr;
        const float* ssq_in = nullptr;
        float* copy_out = nullptr;
        if (head) {
          e.out = a.logits; e.ldo = md.V;
          norm_w = md.final_norm;
          // head-only launches get the residual stream itself as rows and normalise it on load
          if (PRE && n_layers_run > 0) ssq_in = md.ssq;
          else if (head_only) src = src_in;
        } else {
          const LayerDev& ly = layers[l];
          if (which == 0) {          // QKV + RoPE + KV append
            e.qbuf = md.qbuf; e.d = d; e.dh = md.dh; e.max_seq = md.max_seq; e.rowslot = ctl->rowslot; e.rowpos = ctl->rowpos;
            e.cs = md.rope_cos; e.sn = md.rope_sin;
            e.kc = static_cast<WT*>(md.kcache) + (size_t)l * md.max_seq * d;
            e.vc = static_cast<WT*>(md.vcache) + (size_t)l * md.max_seq * d;
            norm_w = ly.attn_norm;
            if (l == 0) { src = src_in; if (cta == 0) copy_out = md.x; }
            else if (PRE) ssq_in = md.ssq;
          } else if (which == 1) {   // output projection + residual
            e.out = md.x; e.ldo = d;
            src = XSrc{md.attn, (size_t)d, nullptr};
            if (PRE) { e.next_gain = ly.ffn_norm; e.xg = md.xg; e.ssq = md.ssq; }
          } else if (which == 2) {   // gate/up + SwiGLU
            e.out = md.act; e.ldo = f;
            norm_w = ly.ffn_norm;
            if (PRE) ssq_in = md.ssq;
          } else {                   // down projection + residual
            e.out = md.x; e.ldo = d;
            src = XSrc{md.act, (size_t)f, nullptr};
            if (PRE) {
              e.next_gain = l + 1 < md.L ? layers[l + 1].attn_norm : md.final_norm;
              e.xg = md.xg; e.ssq = md.ssq;
            }
          }
        }
        consume_gemm<M, WT, TRACE>(g, e, src, norm_w, md.eps, copy_out, ssq_in, cta, G, ring, ctl, X, xphase, red, pre_s,
                            zero_addr, stages, err);
        stamp(3); sync_grid(); stamp(4);
        if (!head && which == 0) {
          if constexpr (sizeof(WT) == 2) attn_phase_mma<M>(md, l, origin, nslots, cta, G, reinterpret_cast<char*>(X), x_bytes(M), ctl);
          else attn_phase<M, WT>(md, l, origin, nslots, cta, G, reinterpret_cast<char*>(X), x_bytes(M), ctl);
          stamp(3); sync_grid(); stamp(4);
        }
      }
      if (want_head) {
        // row statistics over vocabulary slices, then CTA 0 applies the sampling rule
        stats_phase<M>(a.logits, md.V, a.stat_r0, a.stat_n, a.temperature, cta, G, md.stat_part, ctl);
        stamp(3); sync_grid(); stamp(4);
        if (cta == 0 && a.greedy && !a.tree) {
          if (a.mode == MODE_VERIFY) verify_greedy<M>(a, md, st, ctl, G, 0, a.gamma, ctl->tok + 1, pending);
          else if (a.mode == MODE_DRAFT) draft_greedy<M>(a, md, st, ctl, G);
          else verify_greedy<M>(a, md, st, ctl, G, M - 1, 0, ctl->tok, 0);
        }
        stamp();
      }
      if (cta == 0 && tid == 0) {
        if (a.mode == MODE_VERIFY) st->t_verify1 = globaltimer();
        else if (a.mode == MODE_DRAFT) st->t_draft1 = globaltimer();
      }
    }
  }
  __syncthreads();
  if (*err != DEV_OK) {
    // a wait gave up: let copies that are still in flight land before the CTA retires
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  // no member of a cluster retires while another may still arrive on its barrier word
  if (a.cluster_ctas) cluster_sync_all_threads();
}

// ------------------------------------------------------------------------------ bounded waits, exercised
// Runs the two wait primitives of the forward kernel on conditions that never come true, with a
// small poll limit, so that the give-up path (sticky error word, normal return) can be checked on
// a healthy device: which = 0 waits for a phase of a shared-memory barrier nobody arrives at,
// which = 1 enters a grid barrier whose target is one arrival more than the grid will ever make.
// Nothing here can wait longer than `limit` polls.
__global__ void __launch_bounds__(CONSUMER_THREADS) wait_selftest_kernel(DevState* st, unsigned* bar, int which,
                                                                         unsigned limit) {
  __shared__ uint64_t never;
  volatile int* err = &st->err;
  if (threadIdx.x == 0) { mbar_init(&never, 1); mbar_fence_init(); }
  __syncthreads();
  if (which == 0) {
    if (threadIdx.x < 32) mbar_wait(&never, 0u, err, DEV_TIMEOUT_FULL, limit);
  } else {
    unsigned target = 1;   // grid_barrier adds G: G arrivals can never reach G + 1
    grid_barrier(bar, target, gridDim.x, err, limit);
  }
}

// ------------------------------------------------------------------------------ sampling kernels
// Speculative sampling proper (Sec. 2.1 / Sec. 3; p = target, q = draft): accept x_j iff
// u_j < min(1, p_j(x_j) / q_j(x_j)); the first rejected token is replaced by a draw from
// max(0, p_r - q_r) / sum, and if none is rejected a bonus token is drawn from p_{gamma+1}.
// The work that touches a whole vocabulary row is spread over the grid, in two small launches
// behind the forward kernel (which has left the logits and the per-slice row statistics):
//   sample_slices_kernel  every CTA merges the row statistics, repeats the (cheap, deterministic)
//                         accept tests to find r, and reduces its contiguous vocabulary slice of
//                         the weights the next token is drawn from to an integer mass; a draft
//                         step also writes its slice of q_j = softmax(logits / T);
//   sample_pick_kernel    one CTA finds the slice and the token, and commits the step.
// They are separate kernels, not phases of the forward kernel, because that kernel's weight
// streaming loop lost 1.5-2 % of its speed whenever this code was compiled into it.

struct SampleShared {
  float rowmax[MAX_M], rowsum[MAX_M];
  int arg[MAX_M];
  SampleScratch sc;
};

struct SamplePlan {
  int r0, gamma;  // first row and number of draft tokens
  int r;          // accepted draft tokens = row the next token is drawn from
  const float* u; // uniforms of this step: gamma accept tests, then the draw
};

__device__ __forceinline__ const float* step_uniforms(const StepArgs& a, const DevState* st) {
  const float* u = a.uniforms + (a.u_by_block ? (size_t)st->block * a.u_stride : 0);
  return (a.mode == MODE_VERIFY && a.u_by_block) ? u + a.gamma : u;
}

// Every thread of every CTA computes the same plan (same inputs, same arithmetic).
__device__ SamplePlan sample_plan(const StepArgs& a, const DevState* st, SampleShared* sh, int G) {
  const int V = a.md.V;
  SamplePlan pl;
  pl.gamma = a.mode == MODE_VERIFY ? a.gamma : 0;
  pl.r0 = a.mode == MODE_VERIFY ? 0 : a.sample_r0;
  pl.u = step_uniforms(a, st);
  merge_stats(a.md.stat_part, a.fwd_grid, pl.gamma + 1, nullptr, sh->rowmax, sh->rowsum, sh->arg);
  pl.r = pl.gamma;
  for (int j = 0; j < pl.gamma; ++j) {
    int x = st->d_ids[j];
    if ((unsigned)x >= (unsigned)V) x = 0;   // the forward kernel has flagged it; stay in bounds
    const float p = prob_of(ldcg(a.logits + (size_t)(pl.r0 + j) * V + x), a.temperature, sh->rowmax[j], sh->rowsum[j]);
    const float q = ldcg(a.q_in + (size_t)j * V + x);
    if (!accept_test(pl.u[j], p, q)) { pl.r = j; break; }
  }
  return pl;
}

// Calls f(weight function) with the weights of the row the next token is drawn from.
template <class F>
__device__ __forceinline__ void with_weights(const StepArgs& a, const SamplePlan& pl, const SampleShared* sh, F f) {
  const int V = a.md.V;
  const float* lrow = a.logits + (size_t)(pl.r0 + pl.r) * V;
  const float mx = sh->rowmax[pl.r], sm = sh->rowsum[pl.r], T = a.temperature;
  if (a.mode == MODE_DRAFT || pl.r == pl.gamma) {
    f([=](int k) { return prob_of(ldcg(lrow + k), T, mx, sm); });
  } else {
    const float* qrow = a.q_in + (size_t)pl.r * V;
    f([=](int k) { return fmaxf(0.0f, __fsub_rn(prob_of(ldcg(lrow + k), T, mx, sm), ldcg(qrow + k))); });
  }
}

__global__ void __launch_bounds__(SAMPLE_THREADS) sample_slices_kernel(const __grid_constant__ StepArgs a) {
  __shared__ SampleShared sh;
  const int cta = blockIdx.x, G = gridDim.x, V = a.md.V;
  const SamplePlan pl = sample_plan(a, a.st, &sh, G);
  if (cta == 0 && threadIdx.x == 0) {   // the plan travels to the pick kernel behind the slice masses
    __stcg(a.md.cdf_part + 2 * G, (unsigned long long)pl.r);
    __stcg(a.md.cdf_part + 2 * G + 1,
           ((unsigned long long)__float_as_uint(sh.rowmax[pl.r]) << 32) | __float_as_uint(sh.rowsum[pl.r]));
  }
  with_weights(a, pl, &sh, [&](auto wf) {
    if (a.mode == MODE_DRAFT) {   // this CTA's slice of q_j
      float* qrow = a.q_out + (size_t)a.j * V;
      const int VS = (V + G - 1) / G;
      const int k0 = cta * VS, k1 = min(V, k0 + VS);
      for (int k = k0 + threadIdx.x; k < k1; k += SAMPLE_THREADS) stcg(qrow + k, wf(k));
    }
    slice_mass(wf, V, cta, G, a.md.cdf_part, &sh.sc);
  });
}

// One CTA; G = number of slices = the grid of the two kernels before it.
__global__ void __launch_bounds__(SAMPLE_THREADS) sample_pick_kernel(const __grid_constant__ StepArgs a, int G) {
  __shared__ SampleShared sh;
  DevState* st = a.st;
  SamplePlan pl;   // r and the statistics of row r as the slices kernel found them
  pl.gamma = a.mode == MODE_VERIFY ? a.gamma : 0;
  pl.r0 = a.mode == MODE_VERIFY ? 0 : a.sample_r0;
  pl.u = step_uniforms(a, st);
  pl.r = (int)__ldcg(a.md.cdf_part + 2 * G);
  if (pl.r < 0 || pl.r > pl.gamma) pl.r = pl.gamma;
  if (threadIdx.x == 0) {
    const unsigned long long ms = __ldcg(a.md.cdf_part + 2 * G + 1);
    sh.rowmax[pl.r] = __uint_as_float((unsigned)(ms >> 32));
    sh.rowsum[pl.r] = __uint_as_float((unsigned)ms);
  }
  named_sync(1, SAMPLE_THREADS);
  int tok = 0;
  with_weights(a, pl, &sh, [&](auto wf) {
    tok = pick_from_slices(wf, a.md.V, G, a.md.cdf_part, a.mode == MODE_DRAFT ? pl.u[a.j] : pl.u[pl.gamma], &sh.sc);
  });
  if (threadIdx.x == 0) {
    if (a.mode == MODE_DRAFT) {
      st->d_ids[a.j] = tok;
      st->t_draft1 = globaltimer();
    } else {
      commit_step(a, st, pl.r, tok, st->d_ids, st->pending);
      if (a.mode == MODE_VERIFY) st->t_verify1 = globaltimer();
    }
  }
}

// ------------------------------------------------------------------------------ top-k / top-p on the decoding path
// With truncation switched on (Sec. 4 "Decoding" names sampling with top-p / top-k as future work) the
// draw needs whole probability rows: the target's rows p_j and the draft's rows q_j are truncated
// and renormalised (truncate_rows_kernel) and the unchanged rule of Sec. 2.1 runs on those rows.
//   prob_rows_kernel    every CTA merges the row statistics and writes its vocabulary slice of
//                       softmax(logits / T) for the rows the step needs -> prow [rows][V];
//   (truncate_rows_kernel in place on prow)
//   sample_rows_kernel  one CTA: draft step -> x_j drawn from the truncated row, which is also
//                       stored as q_j; verify step -> the rule on (prow, q_in), commit; prefill ->
//                       the first token drawn from the truncated row.

__global__ void __launch_bounds__(SAMPLE_THREADS) prob_rows_kernel(const __grid_constant__ StepArgs a, float* prow) {
  __shared__ SampleShared sh;
  const int cta = blockIdx.x, G = gridDim.x, V = a.md.V;
  const int nrows = a.stat_n, r0 = a.stat_r0;
  // the statistics of row r0 + r sit at index r
  merge_stats(a.md.stat_part, a.fwd_grid, nrows, nullptr, sh.rowmax, sh.rowsum, sh.arg);
  const int VS = (V + G - 1) / G;
  const int k0 = cta * VS, k1 = min(V, k0 + VS);
  for (int r = 0; r < nrows; ++r) {
    const float* lrow = a.logits + (size_t)(r0 + r) * V;
    const float mx = sh.rowmax[r], sm = sh.rowsum[r];
    for (int k = k0 + threadIdx.x; k < k1; k += SAMPLE_THREADS)
      stcg(prow + (size_t)r * V + k, prob_of(ldcg(lrow + k), a.temperature, mx, sm));
  }
}

__global__ void __launch_bounds__(SAMPLE_THREADS) sample_rows_kernel(const __grid_constant__ StepArgs a,
                                                                     const float* prow) {
  __shared__ SampleScratch sc;
  __shared__ int s_ids[MAX_M];
  DevState* st = a.st;
  const int V = a.md.V;
  const float* u = step_uniforms(a, st);
  if (a.mode == MODE_VERIFY) {
    if (threadIdx.x < a.gamma) {
      const int x = st->d_ids[threadIdx.x];
      s_ids[threadIdx.x] = (unsigned)x < (unsigned)V ? x : 0;   // the forward kernel has flagged it
    }
    named_sync(1, SAMPLE_THREADS);
    int r, tok;
    reject_rule_block(prow, a.q_in, s_ids, u, a.gamma, V, 0, &sc, r, tok);
    if (threadIdx.x == 0) {
      commit_step(a, st, r, tok, st->d_ids, st->pending);
      st->t_verify1 = globaltimer();
    }
  } else {
    const int tok = block_sample([&](int k) { return ldcg(prow + k); }, V, a.mode == MODE_DRAFT ? u[a.j] : u[0], &sc);
    if (a.mode == MODE_DRAFT) {
      float* qrow = a.q_out + (size_t)a.j * V;
      for (int k = threadIdx.x; k < V; k += SAMPLE_THREADS) stcg(qrow + k, ldcg(prow + k));
      if (threadIdx.x == 0) { st->d_ids[a.j] = tok; st->t_draft1 = globaltimer(); }
    } else if (threadIdx.x == 0) {
      commit_step(a, st, 0, tok, st->d_ids, st->pending);
    }
  }
}

}  // namespace spd
