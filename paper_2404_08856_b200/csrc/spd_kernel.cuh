// The persistent forward kernel: see spd_engine.cuh for the design.
#pragma once
#include "spd_engine.cuh"

namespace spd {

// Verification (Sec. 2.1 / Sec. 3; p = target, q = draft), run by CTA 0 after the row
// statistics are merged.  Rows r0..r0+gamma of `logits` are p_1..p_{gamma+1}.
template <int M>
__device__ void verify_sample(const StepArgs& a, const ModelDev& md, DevState* st, Ctrl* ctl, int G, int r0,
                              int gamma, const float* u, const int* ids /*gamma draft ids*/, int pending) {
  const int tid = threadIdx.x;
  const int V = md.V;
  float* rmax = ctl->rowmax;
  float* rsum = ctl->rowsum;
  int* rarg = ctl->sc.aidx;
  __shared__ int s_arg[MAX_M];
  merge_stats(md.stat_part, G, gamma + 1, ctl, rmax, rsum, s_arg);
  (void)rarg;
  int r = gamma, tok;
  if (a.greedy) {
    for (int j = 0; j < gamma; ++j)
      if (s_arg[j] != ids[j]) { r = j; break; }
    tok = s_arg[r];
  } else {
    for (int j = 0; j < gamma; ++j) {
      const int x = ids[j];
      const float p = prob_of(ldcg(a.logits + (size_t)(r0 + j) * V + x), a.temperature, rmax[j], rsum[j]);
      const float q = ldcg(a.q_in + (size_t)j * V + x);
      if (!accept_test(u[j], p, q)) { r = j; break; }
    }
    const float* lrow = a.logits + (size_t)(r0 + r) * V;
    const float mx = rmax[r], sm = rsum[r], T = a.temperature;
    if (r < gamma) {
      const float* qrow = a.q_in + (size_t)r * V;
      tok = block_sample(
          [&](int k) { return fmaxf(0.0f, __fsub_rn(prob_of(ldcg(lrow + k), T, mx, sm), ldcg(qrow + k))); }, V,
          u[gamma], &ctl->sc);
    } else {
      tok = block_sample([&](int k) { return prob_of(ldcg(lrow + k), T, mx, sm); }, V, u[gamma], &ctl->sc);
    }
  }
  if (tid == 0) {
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
}

// Draft step j: q_j = softmax(logits/T) written to q_out row j, x_j drawn from it.
template <int M>
__device__ void draft_sample(const StepArgs& a, const ModelDev& md, DevState* st, Ctrl* ctl, int G, int row,
                             const float* u) {
  const int tid = threadIdx.x, V = md.V;
  __shared__ int s_arg[MAX_M];
  // statistics were computed for the single row `row`, stored at index 0
  merge_stats(md.stat_part, G, 1, ctl, ctl->rowmax, ctl->rowsum, s_arg);
  int tok;
  if (a.greedy) {
    tok = s_arg[0];
  } else {
    const float* lrow = a.logits + (size_t)row * V;
    const float mx = ctl->rowmax[0], sm = ctl->rowsum[0], T = a.temperature;
    float* qrow = a.q_out + (size_t)a.j * V;
    for (int k = tid; k < V; k += CONSUMER_THREADS) stcg(qrow + k, prob_of(ldcg(lrow + k), T, mx, sm));
    tok = block_sample([&](int k) { return prob_of(ldcg(lrow + k), T, mx, sm); }, V, u[a.j], &ctl->sc);
  }
  if (tid == 0) st->d_ids[a.j] = tok;
}

template <int M, typename WT>
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
    unsigned bar_target = 0, xphase = 0;
    if (tid == 0) { ctl->trace = cta == 0 ? a.trace : nullptr; ctl->trace_n = 0; }
    named_sync(1, CONSUMER_THREADS);
    auto stamp = [&](int id = 3) { trace_stamp(ctl, id); };
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
      consume_gemm<M, WT>(g, e, src, nullptr, 0.f, nullptr, nullptr, cta, G, ring, ctl, X, xphase, red, pre_s, zero_addr, stages, err);
    } else {
      // positions and token ids of the M rows
      int pos0, pending = 0;
      int ids[M];
      if (a.mode == MODE_VERIFY) {
        pos0 = a.pos_base + st->n_text;
        pending = st->pending;
        ids[0] = pending;
#pragma unroll
        for (int m = 1; m < M; ++m) ids[m] = st->d_ids[m - 1];
      } else if (a.mode == MODE_DRAFT) {
        // rows [token before, token to extend]: tokens are prev, pending, x_1, x_2, ...
        pos0 = a.pos_base + st->n_text - 1 + a.j;
        pending = st->pending;
#pragma unroll
        for (int m = 0; m < M; ++m) {
          const int t = a.j - (M - 1) + m;   // index into [pending, x_1, ...]; -1 = prev
          ids[m] = t < 0 ? st->prev : (t == 0 ? st->pending : st->d_ids[t - 1]);
        }
      } else {
        pos0 = a.rows_pos0;
#pragma unroll
        for (int m = 0; m < M; ++m) ids[m] = a.row_ids ? a.row_ids[m] : 0;
      }
      const bool from_ids = (a.mode != MODE_ROWS) || a.rows == nullptr;
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
        for (int m = 0; m < M; ++m) ctl->tok[m] = ids[m];
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
            e.qbuf = md.qbuf; e.d = d; e.dh = md.dh; e.pos0 = pos0; e.cs = md.rope_cos; e.sn = md.rope_sin;
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
        consume_gemm<M, WT>(g, e, src, norm_w, md.eps, copy_out, ssq_in, cta, G, ring, ctl, X, xphase, red, pre_s,
                            zero_addr, stages, err);
        stamp(3); grid_barrier(a.bar, bar_target, G, err); stamp(4);
        if (!head && which == 0) {
          if constexpr (sizeof(WT) == 2) attn_phase_mma<M>(md, l, pos0, cta, G, reinterpret_cast<char*>(X), x_bytes(M), ctl);
          else attn_phase<M, WT>(md, l, pos0, cta, G, reinterpret_cast<char*>(X), x_bytes(M), ctl);
          stamp(3); grid_barrier(a.bar, bar_target, G, err); stamp(4);
        }
      }
      if (want_head) {
        // row statistics over vocabulary slices, then CTA 0 applies the sampling rule
        int r0, nrows;
        if (a.mode == MODE_VERIFY) { r0 = 0; nrows = a.gamma + 1; }
        else { r0 = M - 1; nrows = 1; }
        stats_phase<M>(a.logits, md.V, r0, nrows, a.temperature, cta, G, md.stat_part, ctl);
        stamp(3); grid_barrier(a.bar, bar_target, G, err); stamp(4);
        if (cta == 0) {
          const float* u = a.uniforms ? a.uniforms + (a.u_by_block ? (size_t)st->block * a.u_stride : 0) : nullptr;
          if (a.mode == MODE_VERIFY) {
            verify_sample<M>(a, md, st, ctl, G, 0, a.gamma, u ? u + (a.u_by_block ? a.gamma : 0) : nullptr, ctl->tok + 1,
                             pending);
          } else if (a.mode == MODE_DRAFT) {
            draft_sample<M>(a, md, st, ctl, G, M - 1, u);
          } else {
            verify_sample<M>(a, md, st, ctl, G, M - 1, 0, u, ctl->tok, 0);
          }
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
}

}  // namespace spd
