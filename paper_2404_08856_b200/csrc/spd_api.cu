// Host side of the C ABI declared in include/spd.h: context, weight repacking, launches.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <string>
#include <vector>

#include "../../include/spd.h"
#include "spd_kernel.cuh"
#include "spd_prefill.cuh"
#include "spd_warp.cuh"
#include "spd_tree.cuh"
#include "spd_batch.cuh"

using namespace spd;

// ------------------------------------------------------------------------------ helpers

namespace {

struct ModelHost {
  spd_model_cfg cfg{};
  ModelDev md{};            // host copy of the device descriptor
  LayerDev* layers_dev = nullptr;
  int pos_base = 0;         // rows in front of the text (image rows / adapter rows)
  float* logits = nullptr;  // [8][V]
  void* adapter = nullptr;  // draft only [d][adapter_in]
  size_t wbytes = 0;        // bytes of matrices streamed per forward (layers + LM head)
  size_t esz = 2;
  // bf16 models: plain row-major copies for the tensor-core prefill (natural row order)
  struct RowMajor { __nv_bfloat16 *wqkv, *wo, *wgu, *wd; const float *attn_norm, *ffn_norm; };
  std::vector<RowMajor> rm;
  __nv_bfloat16* adapter_rm = nullptr;
  __nv_bfloat16* lm_rm = nullptr;   // LM head [V][d], row-major (batched path)
  bool rows_given = false;  // draft only: the image rows arrive already in the draft's space
  int grid = 0;             // CTAs of this model's forward launches (its weights are packed for that count)
  int cluster = 0;          // > 0: those CTAs form one thread-block cluster of this size
};

}  // namespace

struct spd_ctx {
  spd_cfg cfg{};
  cudaStream_t stream = nullptr;
  int device = 0, n_sm = 0, smem_optin = 0;
  ModelHost target, draft;
  DevState* st = nullptr;
  unsigned* bars = nullptr;     // pool of grid-barrier counters
  int bar_next = 0;
  float* ubuf = nullptr;        // [16] uniforms of direct calls: [0..7] draft, [8..15] verify
  float* qbuf = nullptr;        // [gamma_max][V] draft distributions
  float* prow = nullptr;        // [MAX_M][V] probability rows of the step being sampled (top-k / top-p only)
  bool truncate = false;        // top-k / top-p switched on
  // tree blocks (spd_draft_tree / spd_verify_tree): scratch allocated on first use
  float* tree_cur = nullptr;    // [V] renormalised residual between sibling candidates
  char *tree_stage_t = nullptr, *tree_stage_d = nullptr;   // K/V rows in flight during compaction
  TreeShape tree_shape{};       // shape of the last spd_draft_tree
  bool tree_drafted = false;
  float* rows = nullptr;        // prefill rows staging [max_seq][d_max]
  int* ids_dev = nullptr;       // prompt ids [max_seq]
  float* upool = nullptr; size_t upool_cap = 0;
  int* out_dev = nullptr; int out_cap = 0;
  DevState* st_host = nullptr;  // pinned
  std::vector<void*> allocs;
  std::string err;
  bool prefilled = false;
  int drafted_gamma = -1;       // gamma of the last spd_draft not yet verified
  int len_ub = 0;               // upper bound of n_text known to the host
  int n_prompt = 0, m_image = 0;
  int last_verify_rows = 0, last_draft_rows = 0;
  // scratch of the tensor-core prefill, grown on demand
  struct {
    size_t cap_rows = 0;
    __nv_bfloat16 *h_hi = nullptr, *h_lo = nullptr, *q_hi = nullptr, *q_lo = nullptr, *vT = nullptr;
    __nv_bfloat16 *p_hi = nullptr, *p_lo = nullptr;
    __nv_bfloat16 *g_hi = nullptr, *g_lo = nullptr;   // silu(gate) * up [rows][d_ffn]
    float *wide = nullptr, *S = nullptr;
  } pf;
  // scratch of spd_image_adapter, grown on demand
  struct {
    size_t cap_in = 0, cap_hid = 0;      // elements
    float* feats = nullptr;              // staging for host features
    __nv_bfloat16 *f_hi = nullptr, *f_lo = nullptr, *g_hi = nullptr, *g_lo = nullptr;
  } ia;
  cudaStream_t gs = nullptr;             // internal stream: block graphs are captured and replayed here
  cudaGraphExec_t block_exec = nullptr;  // one speculative block (gamma draft steps + verify)
  int block_gamma = -1;
  const float* block_upool = nullptr;
  bool graphs_ok = true;
  unsigned long long* trace = nullptr;   // device buffer of phase timestamps (verify steps)
  int trace_cap = 0;
  cudaEvent_t ev[4]{};
  // spd_fork: a fork shares its origin's weights; the origin is kept alive until the last fork is gone
  spd_ctx* origin = nullptr;
  int n_forks = 0;
  bool zombie = false;       // destroyed by the caller while forks were alive
};

namespace {

constexpr int BAR_POOL = 64;

spd_status fail(spd_ctx* c, spd_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}
#define CU(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess)                                                                    \
      return fail(ctx, e_ == cudaErrorMemoryAllocation ? SPD_ENOMEM : SPD_ECUDA,              \
                  std::string(#call) + ": " + cudaGetErrorString(e_));                        \
  } while (0)

bool is_device_ptr(const void* p) {
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
  return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

template <typename T>
spd_status dalloc(spd_ctx* ctx, T** p, size_t n) {
  void* q = nullptr;
  CU(cudaMalloc(&q, n * sizeof(T) + 256));
  CU(cudaMemsetAsync(q, 0, n * sizeof(T) + 256, ctx->stream));
  ctx->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return SPD_OK;
}

// dst row = map(src row) * dst_mul + dst_off; qk_dh > 0 interleaves rotary pairs:
// source row h*dh + i + w*dh/2 goes to h*dh + 2i + w, so a thread that owns two
// consecutive rows owns one (i, i + dh/2) pair.
__global__ void copy_rows_kernel(char* dst, const char* src, int nrows, int row_bytes, int dst_mul, int dst_off,
                                 int qk_dh) {
  const int chunks = row_bytes >> 4;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)nrows * chunks;
       i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / chunks), c = (int)(i - (size_t)r * chunks);
    int dr = r;
    if (qk_dh > 0) {
      const int h = r / qk_dh, e = r - h * qk_dh, half = qk_dh >> 1;
      dr = h * qk_dh + ((e < half) ? 2 * e : 2 * (e - half) + 1);
    }
    dr = dr * dst_mul + dst_off;
    reinterpret_cast<uint4*>(dst + (size_t)dr * row_bytes)[c] =
        reinterpret_cast<const uint4*>(src + (size_t)r * row_bytes)[c];
  }
}

spd_status put_rows(spd_ctx* ctx, void* dst, const void* src, void* staging, int nrows, int rowlen, size_t esz,
                    int dst_mul, int dst_off, int qk_dh) {
  if (!src) return fail(ctx, SPD_EINVAL, "missing weight pointer");
  const size_t bytes = (size_t)nrows * rowlen * esz;
  CU(cudaMemcpyAsync(staging, src, bytes, cudaMemcpyDefault, ctx->stream));
  copy_rows_kernel<<<1184, 256, 0, ctx->stream>>>(static_cast<char*>(dst), static_cast<const char*>(staging), nrows,
                                                  (int)(rowlen * esz), dst_mul, dst_off, qk_dh);
  CU(cudaGetLastError());
  CU(cudaStreamSynchronize(ctx->stream));  // staging is reused; host sources may be pageable
  return SPD_OK;
}

// Row-major [N][K] -> the streaming layout of spd_engine.cuh: rows dealt to the G CTAs in
// quads, each CTA's rows cut into tiles of up to 32 rows, a tile stored step by step
// ([step][row][512 B]); zero padding for rows >= N and columns >= K; for 2-byte elements the
// 16-byte chunks of a row are XOR-swizzled with (row-in-tile & 7).
__global__ void pack_tiles_kernel(char* dst, const char* src, int N, int K, int esz, int G) {
  const int kstep = 512 / esz, nsteps = (K + kstep - 1) / kstep, epc = 16 / esz;
  const long long Q = (N + 3) >> 2;
  const size_t total = (size_t)Q * 4 * nsteps * 32;   // 16-byte chunks
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int kc = (int)(i & 31);
    const size_t rs = i >> 5;
    const int s = (int)(rs % nsteps), n = (int)(rs / nsteps);
    const long long q = n >> 2;
    int c = (int)(((q + 1) * G + Q - 1) / Q) - 1;
    while (c > 0 && Q * c / G > q) --c;
    while (c < G - 1 && Q * (c + 1) / G <= q) ++c;
    const int q0 = (int)(Q * c / G), q1 = (int)(Q * (c + 1) / G);
    const int rl = n - q0 * 4, t = rl >> 5, ri = rl & 31;
    const int nr = min(32, (q1 - q0) * 4 - t * 32);
    const int phys = esz == 2 ? (kc ^ (ri & 7)) : kc;
    const int k = s * kstep + kc * epc;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (n < N && k < K) v = *reinterpret_cast<const uint4*>(src + ((size_t)n * K + k) * esz);
    const size_t off = (((size_t)(q0 * 4 + t * 32) * nsteps + (size_t)s * nr + ri) * 512) + (size_t)phys * 16;
    *reinterpret_cast<uint4*>(dst + off) = v;
  }
}

__global__ void widen_bf16_kernel(float* dst, const uint16_t* src, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = __uint_as_float((uint32_t)src[i] << 16);
}

size_t packed_bytes(int N, int K, size_t esz) {
  const int kstep = (int)(512 / esz);
  return (size_t)((N + 3) / 4) * 4 * ((K + kstep - 1) / kstep) * 512;
}

spd_status pack_tiles(spd_ctx* ctx, void* dst, const void* src_rowmajor, int N, int K, size_t esz, int G,
                      cudaStream_t st) {
  pack_tiles_kernel<<<1184, 256, 0, st>>>(static_cast<char*>(dst), static_cast<const char*>(src_rowmajor), N, K,
                                          (int)esz, G);
  CU(cudaGetLastError());
  return SPD_OK;
}

spd_status check_model(spd_ctx* ctx, const spd_model_cfg& c, const char* who) {
  auto bad = [&](const char* what) { return fail(ctx, SPD_EINVAL, std::string(who) + ": " + what); };
  if (c.n_layers < 1 || c.d_model < 8 || c.n_heads < 1 || c.d_ffn < 8 || c.vocab < 2) return bad("non-positive shape");
  if (c.d_model % c.n_heads) return bad("d_model not divisible by n_heads");
  const int dh = c.d_model / c.n_heads;
  if (dh != 32 && dh != 64 && dh != 128) return bad("d_head must be 32, 64 or 128");
  // the tensor-core attention tiles swizzle the eight 16-byte pieces of a 128-byte row segment: a
  // bf16 row needs at least eight pieces
  if (c.dtype == 1 && dh == 32) return bad("bf16 models need d_head 64 or 128");
  if (c.d_model > KC_MAX) return bad("d_model > 4096 not supported");
  if (c.d_model % 32 || c.d_ffn % 8) return bad("d_model must be a multiple of 32 and d_ffn of 8");
  if (c.dtype != 0 && c.dtype != 1) return bad("dtype must be 0 (fp32) or 1 (bf16)");
  if (!(c.rms_eps >= 0.f) || !(c.rope_theta > 0.f)) return bad("bad rms_eps / rope_theta");
  return SPD_OK;
}

// Everything of a model that belongs to ONE sequence: KV cache, activation rows, attention
// partials, statistics, logits.  (Weights, embedding table, layer records and rotary tables are
// shared between a context and its forks.)
spd_status alloc_sequence_state(spd_ctx* ctx, ModelHost& mh) {
  const spd_model_cfg& c = mh.cfg;
  const int d = c.d_model, f = c.d_ffn, V = c.vocab, L = c.n_layers, H = c.n_heads, dh = d / H;
  const int max_seq = ctx->cfg.max_seq;
  const size_t esz = mh.esz;
  ModelDev& md = mh.md;
  spd_status s;
  char *kc, *vc;
  if ((s = dalloc(ctx, &kc, (size_t)L * max_seq * d * esz))) return s;
  if ((s = dalloc(ctx, &vc, (size_t)L * max_seq * d * esz))) return s;
  md.kcache = kc; md.vcache = vc;
  if ((s = dalloc(ctx, &md.x, (size_t)MAX_M * d))) return s;
  if ((s = dalloc(ctx, &md.qbuf, (size_t)MAX_M * d))) return s;
  if ((s = dalloc(ctx, &md.xg, (size_t)MAX_M * d))) return s;
  if ((s = dalloc(ctx, &md.ssq, (size_t)ctx->n_sm * 8))) return s;
  if ((s = dalloc(ctx, &md.attn, (size_t)MAX_M * d))) return s;
  if ((s = dalloc(ctx, &md.act, (size_t)MAX_M * f))) return s;
  if ((s = dalloc(ctx, &md.apart, (size_t)H * md.nsplit * MAX_M * dh))) return s;
  if ((s = dalloc(ctx, &md.aml, (size_t)H * md.nsplit * MAX_M * 2))) return s;
  if ((s = dalloc(ctx, &md.head_cnt, (size_t)H))) return s;
  if ((s = dalloc(ctx, &md.stat_part, (size_t)ctx->n_sm * MAX_M * 4))) return s;
  if ((s = dalloc(ctx, &md.cdf_part, (size_t)ctx->n_sm * 2 + 2))) return s;
  if ((s = dalloc(ctx, &mh.logits, (size_t)MAX_M * V))) return s;
  return SPD_OK;
}

spd_status build_model(spd_ctx* ctx, ModelHost& mh, const spd_model_cfg& c, const spd_weights* w, int adapter_in,
                       void* staging, char* rm) {
  mh.cfg = c;
  const size_t esz = c.dtype == 1 ? 2 : 4;
  mh.esz = esz;
  const int d = c.d_model, f = c.d_ffn, V = c.vocab, L = c.n_layers, H = c.n_heads, dh = d / H;
  const int max_seq = ctx->cfg.max_seq;
  ModelDev& md = mh.md;
  md.L = L; md.d = d; md.H = H; md.dh = dh; md.f = f; md.V = V; md.max_seq = max_seq;
  md.nsplit = mh.grid / H > 0 ? mh.grid / H : 1;
  md.eps = c.rms_eps;
  md.scale = (float)(1.0 / sqrt((double)dh));
  spd_status s;
  {  // the embedding table is kept in fp32 so that rows can be bulk-copied as activations
    float* embed = nullptr;
    if ((s = dalloc(ctx, &embed, (size_t)V * d))) return s;
    if (!w->tok_embed) return fail(ctx, SPD_EINVAL, "missing tok_embed");
    if (esz == 4) {
      CU(cudaMemcpyAsync(embed, w->tok_embed, (size_t)V * d * 4, cudaMemcpyDefault, ctx->stream));
    } else {
      CU(cudaMemcpyAsync(staging, w->tok_embed, (size_t)V * d * 2, cudaMemcpyDefault, ctx->stream));
      widen_bf16_kernel<<<1184, 256, 0, ctx->stream>>>(embed, reinterpret_cast<const uint16_t*>(staging), (size_t)V * d);
      CU(cudaGetLastError());
    }
    CU(cudaStreamSynchronize(ctx->stream));
    md.embed = embed;
  }
  {  // the LM head is streamed tile-packed; a tied head is a packed copy of the table
    char* lm = nullptr;
    if ((s = dalloc(ctx, &lm, packed_bytes(V, d, esz)))) return s;
    if ((s = put_rows(ctx, rm, c.tied_embeddings ? w->tok_embed : w->lm_head, staging, V, d, esz, 1, 0, 0))) return s;
    if ((s = pack_tiles(ctx, lm, rm, V, d, esz, mh.grid, ctx->stream))) return s;
    md.lm_head = lm;
    if (esz == 2) {   // natural-order copy for the dense (batched) path
      if ((s = dalloc(ctx, &mh.lm_rm, (size_t)V * d))) return s;
      CU(cudaMemcpyAsync(mh.lm_rm, rm, (size_t)V * d * 2, cudaMemcpyDeviceToDevice, ctx->stream));
      CU(cudaStreamSynchronize(ctx->stream));
    }
  }
  float* fn = nullptr;
  if ((s = dalloc(ctx, &fn, (size_t)d))) return s;
  if (!w->final_norm) return fail(ctx, SPD_EINVAL, "missing final_norm");
  CU(cudaMemcpyAsync(fn, w->final_norm, d * sizeof(float), cudaMemcpyDefault, ctx->stream));
  md.final_norm = fn;
  mh.rows_given = adapter_in > 0 && !w->adapter && adapter_in == d;
  if (adapter_in > 0 && !mh.rows_given) {
    if (!w->adapter) return fail(ctx, SPD_EINVAL, "draft_adapter_in > 0 but no adapter weights");
    char* ad = nullptr;
    if ((s = dalloc(ctx, &ad, packed_bytes(d, adapter_in, esz)))) return s;
    if ((s = put_rows(ctx, rm, w->adapter, staging, d, adapter_in, esz, 1, 0, 0))) return s;
    if ((s = pack_tiles(ctx, ad, rm, d, adapter_in, esz, mh.grid, ctx->stream))) return s;
    mh.adapter = ad;
  }
  std::vector<LayerDev> layers(L);
  if (!w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down)
    return fail(ctx, SPD_EINVAL, "missing per-layer weight array");
  for (int l = 0; l < L; ++l) {
    char *wqkv, *wo, *wgu, *wd;
    float *an, *fnw;
    if ((s = dalloc(ctx, &wqkv, packed_bytes(3 * d, d, esz)))) return s;
    if ((s = dalloc(ctx, &wo, packed_bytes(d, d, esz)))) return s;
    if ((s = dalloc(ctx, &wgu, packed_bytes(2 * f, d, esz)))) return s;
    if ((s = dalloc(ctx, &wd, packed_bytes(d, f, esz)))) return s;
    if ((s = dalloc(ctx, &an, (size_t)d))) return s;
    if ((s = dalloc(ctx, &fnw, (size_t)d))) return s;
    // compose the permuted row-major matrix in `rm`, then tile-pack it
    if ((s = put_rows(ctx, rm, w->wq[l], staging, d, d, esz, 1, 0, dh))) return s;
    if ((s = put_rows(ctx, rm + (size_t)d * d * esz, w->wk[l], staging, d, d, esz, 1, 0, dh))) return s;
    if ((s = put_rows(ctx, rm + (size_t)2 * d * d * esz, w->wv[l], staging, d, d, esz, 1, 0, 0))) return s;
    if ((s = pack_tiles(ctx, wqkv, rm, 3 * d, d, esz, mh.grid, ctx->stream))) return s;
    if ((s = put_rows(ctx, rm, w->wo[l], staging, d, d, esz, 1, 0, 0))) return s;
    if ((s = pack_tiles(ctx, wo, rm, d, d, esz, mh.grid, ctx->stream))) return s;
    if ((s = put_rows(ctx, rm, w->w_gate[l], staging, f, d, esz, 2, 0, 0))) return s;
    if ((s = put_rows(ctx, rm, w->w_up[l], staging, f, d, esz, 2, 1, 0))) return s;
    if ((s = pack_tiles(ctx, wgu, rm, 2 * f, d, esz, mh.grid, ctx->stream))) return s;
    if ((s = put_rows(ctx, rm, w->w_down[l], staging, d, f, esz, 1, 0, 0))) return s;
    if ((s = pack_tiles(ctx, wd, rm, d, f, esz, mh.grid, ctx->stream))) return s;
    if (!w->attn_norm[l] || !w->ffn_norm[l]) return fail(ctx, SPD_EINVAL, "missing norm gain");
    CU(cudaMemcpyAsync(an, w->attn_norm[l], d * sizeof(float), cudaMemcpyDefault, ctx->stream));
    CU(cudaMemcpyAsync(fnw, w->ffn_norm[l], d * sizeof(float), cudaMemcpyDefault, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    layers[l] = LayerDev{wqkv, wo, wgu, wd, an, fnw};
    if (esz == 2) {   // natural-order copies for the prefill GEMMs
      ModelHost::RowMajor r{};
      if ((s = dalloc(ctx, &r.wqkv, (size_t)3 * d * d))) return s;
      if ((s = dalloc(ctx, &r.wo, (size_t)d * d))) return s;
      if ((s = dalloc(ctx, &r.wgu, (size_t)2 * f * d))) return s;
      if ((s = dalloc(ctx, &r.wd, (size_t)d * f))) return s;
      CU(cudaMemcpyAsync(r.wqkv, w->wq[l], (size_t)d * d * 2, cudaMemcpyDefault, ctx->stream));
      CU(cudaMemcpyAsync(r.wqkv + (size_t)d * d, w->wk[l], (size_t)d * d * 2, cudaMemcpyDefault, ctx->stream));
      CU(cudaMemcpyAsync(r.wqkv + (size_t)2 * d * d, w->wv[l], (size_t)d * d * 2, cudaMemcpyDefault, ctx->stream));
      CU(cudaMemcpyAsync(r.wo, w->wo[l], (size_t)d * d * 2, cudaMemcpyDefault, ctx->stream));
      // gate and up rows interleaved (gate_0, up_0, gate_1, ...): the GEMM's epilogue pairs them
      if ((s = put_rows(ctx, r.wgu, w->w_gate[l], staging, f, d, esz, 2, 0, 0))) return s;
      if ((s = put_rows(ctx, r.wgu, w->w_up[l], staging, f, d, esz, 2, 1, 0))) return s;
      CU(cudaMemcpyAsync(r.wd, w->w_down[l], (size_t)d * f * 2, cudaMemcpyDefault, ctx->stream));
      CU(cudaStreamSynchronize(ctx->stream));
      r.attn_norm = an; r.ffn_norm = fnw;
      mh.rm.push_back(r);
    }
  }
  if (esz == 2 && adapter_in > 0 && !mh.rows_given) {
    if ((s = dalloc(ctx, &mh.adapter_rm, (size_t)d * adapter_in))) return s;
    CU(cudaMemcpyAsync(mh.adapter_rm, w->adapter, (size_t)d * adapter_in * 2, cudaMemcpyDefault, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
  }
  if ((s = dalloc(ctx, &mh.layers_dev, (size_t)L))) return s;
  CU(cudaMemcpyAsync(mh.layers_dev, layers.data(), L * sizeof(LayerDev), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  md.layers = mh.layers_dev;
  // rotary table: cos/sin(pos * theta^(-2i/dh)) in double, stored fp32
  {
    const int half = dh / 2;
    std::vector<float> cs((size_t)max_seq * half), sn((size_t)max_seq * half);
    for (int i = 0; i < half; ++i) {
      const double inv = pow((double)c.rope_theta, -2.0 * i / (double)dh);
      for (int p = 0; p < max_seq; ++p) {
        cs[(size_t)p * half + i] = (float)cos(p * inv);
        sn[(size_t)p * half + i] = (float)sin(p * inv);
      }
    }
    float *dc, *ds;
    if ((s = dalloc(ctx, &dc, cs.size()))) return s;
    if ((s = dalloc(ctx, &ds, sn.size()))) return s;
    CU(cudaMemcpyAsync(dc, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(ds, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    md.rope_cos = dc; md.rope_sin = ds;
  }
  if ((s = alloc_sequence_state(ctx, mh))) return s;
  CU(cudaStreamSynchronize(ctx->stream));
  mh.wbytes = ((size_t)L * (4ull * d * d + 3ull * d * f) + (size_t)V * d) * esz;
  return SPD_OK;
}

// ---- kernel dispatch

using KernelFn = void (*)(const StepArgs);

template <typename WT, bool TRACE>
KernelFn pick_m(int M) {
  switch (M) {
    case 1: return forward_kernel<1, WT, TRACE>;
    case 2: return forward_kernel<2, WT, TRACE>;
    case 3: return forward_kernel<3, WT, TRACE>;
    case 4: return forward_kernel<4, WT, TRACE>;
    case 5: return forward_kernel<5, WT, TRACE>;
    case 6: return forward_kernel<6, WT, TRACE>;
    case 7: return forward_kernel<7, WT, TRACE>;
    default: return forward_kernel<8, WT, TRACE>;
  }
}
// trace: the instantiation with phase timestamps (spd_trace); the plain one carries none
KernelFn pick_kernel(int M, int dtype, bool trace = false) {
  if (trace) return dtype == 1 ? pick_m<__nv_bfloat16, true>(M) : pick_m<float, true>(M);
  return dtype == 1 ? pick_m<__nv_bfloat16, false>(M) : pick_m<float, false>(M);
}

struct LaunchCfg { int nstage; size_t smem; };

constexpr int MAX_DEV = 64;   // devices per process that the per-device tables below cover

spd_status launch_cfg(spd_ctx* ctx, KernelFn fn, int M, int n_sm, int smem_optin, LaunchCfg* lc) {
  // per device and kernel variant; filled on first use (the shared-memory attribute of a kernel
  // belongs to the device it was set on)
  static LaunchCfg cache_all[MAX_DEV][4 * (MAX_M + 1)];
  static KernelFn cache_fn_all[MAX_DEV][4 * (MAX_M + 1)];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return fail(ctx, SPD_ECUDA, "no current device");
  LaunchCfg* cache = cache_all[dev];
  KernelFn* cache_fn = cache_fn_all[dev];
  for (int i = 0; i < 4 * (MAX_M + 1); ++i)
    if (cache_fn[i] == fn) { *lc = cache[i]; return SPD_OK; }
  cudaFuncAttributes fa{};
  CU(cudaFuncGetAttributes(&fa, (const void*)fn));
  const size_t fixed = FIXED_SMEM + (size_t)x_bytes(M);
  const size_t avail = (size_t)smem_optin - fa.sharedSizeBytes;
  if (avail < fixed + 2 * STAGE_BYTES) return fail(ctx, SPD_ECUDA, "not enough shared memory per block");
  int ns = (int)((avail - fixed) / STAGE_BYTES);
  if (ns > NSTAGE_MAX) ns = NSTAGE_MAX;
  lc->nstage = ns;
  lc->smem = fixed + (size_t)ns * STAGE_BYTES;
  CU(cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lc->smem));
  (void)n_sm;
  for (int i = 0; i < 4 * (MAX_M + 1); ++i)
    if (!cache_fn[i]) { cache[i] = *lc; cache_fn[i] = fn; break; }
  return SPD_OK;
}

unsigned* next_bar(spd_ctx* ctx);

// One cluster of `cs` CTAs with this kernel's shared memory must be able to run.
bool cluster_fits(KernelFn fn, int cs, size_t smem) {
  if (cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(cs); cfg.blockDim = dim3(ENGINE_THREADS); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, (const void*)fn, &cfg) != cudaSuccess) { cudaGetLastError(); return false; }
  return n >= 1;
}

// grid = CTAs of the launch; cluster > 0: they form one thread-block cluster (then grid == cluster)
// and synchronise inside it, otherwise it is a cooperative launch with the barrier word `bar`.
spd_status launch_forward(spd_ctx* ctx, int M, int dtype, StepArgs a, cudaStream_t stream, int grid, int cluster,
                          int smem_optin, unsigned* bar, int n_sm_sampling) {
  KernelFn fn = pick_kernel(M, dtype, a.trace != nullptr);
  LaunchCfg lc{};
  spd_status s = launch_cfg(ctx, fn, M, grid, smem_optin, &lc);
  if (s) return s;
  a.nstage = lc.nstage;
  a.bar = bar;
  a.cluster_ctas = cluster;
  a.fwd_grid = grid;
  a.sample_r0 = M - 1;
  void* params[] = {&a};
  if (cluster > 0) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(ENGINE_THREADS); cfg.dynamicSmemBytes = lc.smem; cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    CU(cudaLaunchKernelExC(&cfg, (const void*)fn, params));
  } else {
    CU(cudaMemsetAsync(bar, 0, sizeof(unsigned), stream));
    CU(cudaLaunchCooperativeKernel((const void*)fn, dim3(grid), dim3(ENGINE_THREADS), params, lc.smem, stream));
  }
  // sampling (not greedy): the forward kernel has left logits and per-slice row statistics; two
  // small kernels spread the draw over the whole device and commit the step
  const bool samples = a.mode == MODE_VERIFY || a.mode == MODE_DRAFT || (a.mode == MODE_ROWS && a.want_sample);
  if (samples && !a.greedy && !a.tree) {
    if (ctx && ctx->truncate) {
      // top-k / top-p: probability rows -> truncated and renormalised in place -> the rule on rows
      const int nrows = a.mode == MODE_VERIFY ? a.gamma + 1 : 1;
      prob_rows_kernel<<<n_sm_sampling, SAMPLE_THREADS, 0, stream>>>(a, ctx->prow);
      truncate_rows_kernel<<<nrows, WARP_THREADS, (size_t)a.md.V * sizeof(float), stream>>>(
          ctx->prow, ctx->prow, a.md.V, ctx->cfg.top_k, ctx->cfg.top_p > 0.f ? ctx->cfg.top_p : 1.0f);
      sample_rows_kernel<<<1, SAMPLE_THREADS, 0, stream>>>(a, ctx->prow);
    } else {
      sample_slices_kernel<<<n_sm_sampling, SAMPLE_THREADS, 0, stream>>>(a);
      sample_pick_kernel<<<1, SAMPLE_THREADS, 0, stream>>>(a, n_sm_sampling);
    }
    CU(cudaGetLastError());
  }
  return SPD_OK;
}

spd_status launch_model(spd_ctx* ctx, ModelHost& mh, int M, StepArgs a, cudaStream_t stream) {
  return launch_forward(ctx, M, mh.cfg.dtype, a, stream, mh.grid, mh.cluster, ctx->smem_optin, next_bar(ctx), ctx->n_sm);
}

unsigned* next_bar(spd_ctx* ctx) {
  unsigned* b = ctx->bars + 32 * (ctx->bar_next % BAR_POOL);  // 128 B apart
  ctx->bar_next++;
  return b;
}

spd_status check_dev_err(spd_ctx* ctx, int e) {
  if (e == DEV_OK) return SPD_OK;
  if (e == DEV_BAD_TOKEN) return fail(ctx, SPD_EINVAL, "token id out of range seen on the device");
  return fail(ctx, SPD_ETIMEOUT, "device-side wait ran out (code " + std::to_string(e) + ")");
}

spd_status sync_state(spd_ctx* ctx, cudaStream_t stream = nullptr, bool use_given = false) {
  cudaStream_t cs = use_given ? stream : ctx->stream;
  CU(cudaMemcpyAsync(ctx->st_host, ctx->st, sizeof(DevState), cudaMemcpyDeviceToHost, cs));
  CU(cudaStreamSynchronize(cs));
  ctx->len_ub = ctx->st_host->n_text;
  const int e = ctx->st_host->err;
  if (e != DEV_OK) {
    cudaMemsetAsync(&ctx->st->err, 0, sizeof(int), ctx->stream);
    return check_dev_err(ctx, e);
  }
  return SPD_OK;
}

spd_status copy_out(spd_ctx* ctx, void* dst, const void* src_dev, size_t bytes, bool* need_sync) {
  if (!dst) return SPD_OK;
  if (is_device_ptr(dst)) {
    CU(cudaMemcpyAsync(dst, src_dev, bytes, cudaMemcpyDeviceToDevice, ctx->stream));
  } else {
    CU(cudaMemcpyAsync(dst, src_dev, bytes, cudaMemcpyDeviceToHost, ctx->stream));
    *need_sync = true;
  }
  return SPD_OK;
}

// Row tables of the two plain launches (spd_engine.cuh, RowGeom).  Verify: the chain
// [pending, x_1..x_gamma] from the origin on.  Draft step j: the two rows [token before, token to
// extend] at slots j-1 and j (slot -1 is the previous token's row, recomputed identically).
void geom_verify_chain(StepArgs& a, int gamma) {
  for (int m = 0; m <= gamma; ++m) {
    a.geo.slot[m] = a.geo.depth[m] = (signed char)m;
    a.geo.sees[m] = (unsigned char)((2u << m) - 1u);
    a.geo.src[m] = (signed char)(m - 1);
  }
  a.n_slots = gamma + 1;
  a.stat_r0 = 0; a.stat_n = gamma + 1;
}
void geom_draft_step(StepArgs& a, int j) {
  a.geo.slot[0] = a.geo.depth[0] = (signed char)(j - 1);
  a.geo.sees[0] = (unsigned char)((1u << j) - 1u);
  a.geo.src[0] = (signed char)(j == 0 ? -2 : j - 2);
  a.geo.slot[1] = a.geo.depth[1] = (signed char)j;
  a.geo.sees[1] = (unsigned char)((2u << j) - 1u);
  a.geo.src[1] = (signed char)(j - 1);
  a.n_slots = j + 1;
  a.stat_r0 = 1; a.stat_n = 1;
}

StepArgs base_args(spd_ctx* ctx, ModelHost& mh) {
  StepArgs a{};
  a.md = mh.md;
  a.st = ctx->st;
  a.greedy = ctx->cfg.greedy;
  a.temperature = ctx->cfg.temperature;
  a.pos_base = mh.pos_base;
  a.logits = mh.logits;
  return a;
}

// Feed rows [r0, r1) of a prompt through a model in chunks of up to 8 rows.
spd_status feed_rows(spd_ctx* ctx, ModelHost& mh, const float* rows_dev, const int* ids_dev, int r0, int r1,
                     int pos0, bool sample_last, int init_n_text, int init_prev) {
  const int d = mh.cfg.d_model;
  for (int r = r0; r < r1; r += MAX_M) {
    const int M = (r1 - r) < MAX_M ? (r1 - r) : MAX_M;
    StepArgs a = base_args(ctx, mh);
    a.mode = MODE_ROWS;
    a.rows = rows_dev ? rows_dev + (size_t)r * d : nullptr;
    a.row_ids = ids_dev ? ids_dev + r : nullptr;
    a.rows_pos0 = pos0 + (r - r0);
    a.want_sample = sample_last && (r + M >= r1);
    a.stat_r0 = M - 1; a.stat_n = 1;
    a.init_n_text = init_n_text;
    a.init_prev = init_prev;
    a.uniforms = ctx->ubuf + 8;
    a.out_ids = ctx->out_dev;
    spd_status s = launch_model(ctx, mh, M, a, ctx->stream);
    if (s) return s;
  }
  return SPD_OK;
}


// ---- tensor-core prefill (bf16 models)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q{};
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 operand view [batch][rows][inner] with byte strides; box = 64 inner x 128 rows x 1.
spd_status make_map(spd_ctx* ctx, CUtensorMap* m, const void* ptr, int inner, int rows, int batch, size_t row_stride,
                    size_t batch_stride, int box_rows = TC_BM) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return fail(ctx, SPD_ECUDA, "cuTensorMapEncodeTiled not available");
  const cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)batch};
  const cuuint64_t strides[2] = {(cuuint64_t)row_stride, (cuuint64_t)batch_stride};
  const cuuint32_t box[3] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, SPD_ECUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  return SPD_OK;
}

struct Operand { const void* ptr; int inner, rows, batch; size_t row_stride, batch_stride; };

// stream_ksplit = 0: the prefill form (3 stages, two CTAs per SM).  > 0: few rows against a large
// weight matrix -- 6 stages, one CTA per SM, and the K loop cut into that many slices so that
// enough CTAs stream; the slices' partial products go to `ws` and are summed in slice order.
// `wide`: weight-tile rows of the streaming form (0 or 128, 160, 256): the wider, the fewer activation bytes
// re-read per weight byte.
spd_status tc_gemm(spd_ctx* ctx, const Operand& a_hi, const Operand& a_lo, const Operand& b, TcArgs args,
                   bool gelu = false, int stream_ksplit = 0, float* ws = nullptr, int wide = 0,
                   bool leave_slices = false) {
  CUtensorMap ma, ml, mb;
  spd_status s;
  if ((s = make_map(ctx, &ma, a_hi.ptr, a_hi.inner, a_hi.rows, a_hi.batch, a_hi.row_stride, a_hi.batch_stride))) return s;
  if ((s = make_map(ctx, &ml, a_lo.ptr, a_lo.inner, a_lo.rows, a_lo.batch, a_lo.row_stride, a_lo.batch_stride))) return s;
  if ((s = make_map(ctx, &mb, b.ptr, b.inner, b.rows, b.batch, b.row_stride, b.batch_stride,
                    stream_ksplit > 0 && wide > 0 ? wide : TC_BN))) return s;
  static bool attr_set[MAX_DEV];
  if (ctx->device < 0 || ctx->device >= MAX_DEV) return fail(ctx, SPD_ECUDA, "device index out of range");
  if (!attr_set[ctx->device]) {
    CU(cudaFuncSetAttribute((const void*)tc_gemm_kernel<false, TC_STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
    CU(cudaFuncSetAttribute((const void*)tc_gemm_kernel<true, TC_STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
    CU(cudaFuncSetAttribute((const void*)tc_gemm_kernel<false, TC_STAGES_STREAM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            tc_smem_bytes(TC_STAGES_STREAM)));
    CU(cudaFuncSetAttribute((const void*)tc_gemm_kernel<false, TC_STAGES_WIDE, TC_BN_WIDE>,
                            cudaFuncAttributeMaxDynamicSharedMemorySize, tc_smem_bytes(TC_STAGES_WIDE, TC_BN_WIDE)));
    CU(cudaFuncSetAttribute((const void*)tc_gemm_kernel<false, TC_STAGES_MID, TC_BN_MID>,
                            cudaFuncAttributeMaxDynamicSharedMemorySize, tc_smem_bytes(TC_STAGES_MID, TC_BN_MID)));
    attr_set[ctx->device] = true;
  }
  args.split = 1;
  args.err = &ctx->st->err;
  args.ksplit = 1;
  if (stream_ksplit > 0) {
    if (gelu || a_hi.batch != 1 || args.mode == TC_OUT_SPLIT || (args.mode == TC_OUT_SWIGLU && stream_ksplit > 1))
      return fail(ctx, SPD_EINVAL, "streaming GEMM: fp32 output, or the SwiGLU epilogue on an unsliced K");
    const int mode = args.mode;
    float* dest = args.out_f32;
    const long long ldo = args.ldo;
    if (stream_ksplit > 1) {
      if (!ws || ldo != args.N) return fail(ctx, SPD_EINVAL, "split GEMM needs a workspace and a dense output");
      args.ksplit = stream_ksplit; args.out_f32 = ws; args.mode = TC_OUT_F32;
    }
    if (wide != 0 && wide != TC_BN && wide != TC_BN_MID && wide != TC_BN_WIDE) return fail(ctx, SPD_EINVAL, "streaming GEMM: tile width");
    const int bn = wide > 0 ? wide : TC_BN;
    dim3 grid((args.N + bn - 1) / bn, (args.M + TC_BM - 1) / TC_BM, stream_ksplit);
    if (bn == TC_BN_WIDE)
      tc_gemm_kernel<false, TC_STAGES_WIDE, TC_BN_WIDE><<<grid, 128, tc_smem_bytes(TC_STAGES_WIDE, TC_BN_WIDE), ctx->stream>>>(ma, ml, mb, args);
    else if (bn == TC_BN_MID)
      tc_gemm_kernel<false, TC_STAGES_MID, TC_BN_MID><<<grid, 128, tc_smem_bytes(TC_STAGES_MID, TC_BN_MID), ctx->stream>>>(ma, ml, mb, args);
    else
      tc_gemm_kernel<false, TC_STAGES_STREAM><<<grid, 128, tc_smem_bytes(TC_STAGES_STREAM), ctx->stream>>>(ma, ml, mb, args);
    if (stream_ksplit > 1 && !leave_slices)   // (leave_slices: the caller's next kernel adds them up)
      tc_reduce_kernel<<<148, 256, 0, ctx->stream>>>(ws, stream_ksplit, (size_t)args.M * args.N, dest, mode == TC_OUT_F32_ADD);
    CU(cudaGetLastError());
    return SPD_OK;
  }
  dim3 grid((args.N + TC_BN - 1) / TC_BN, (args.M + TC_BM - 1) / TC_BM, a_hi.batch);
  if (gelu) tc_gemm_kernel<true, TC_STAGES><<<grid, 128, TC_SMEM_BYTES, ctx->stream>>>(ma, ml, mb, args);
  else tc_gemm_kernel<false, TC_STAGES><<<grid, 128, TC_SMEM_BYTES, ctx->stream>>>(ma, ml, mb, args);
  CU(cudaGetLastError());
  return SPD_OK;
}

// Embedding rows of n token ids.  An id outside [0, V) (possible when the ids live in device
// memory, which the host cannot inspect) is read as token 0 and recorded in *err.
__global__ void gather_rows_kernel(const int* ids, const float* table, float* out, int n, int d, int V, int* err) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)n * (d >> 2);
       i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / (d >> 2)), c = (int)(i - (size_t)r * (d >> 2));
    int id = ids[r];
    if ((unsigned)id >= (unsigned)V) {
      if (c == 0) atomicCAS(err, DEV_OK, DEV_BAD_TOKEN);
      id = 0;
    }
    reinterpret_cast<float4*>(out + (size_t)r * d)[c] = reinterpret_cast<const float4*>(table + (size_t)id * d)[c];
  }
}

spd_status prefill_scratch(spd_ctx* ctx, int R) {
  if ((size_t)R <= ctx->pf.cap_rows) return SPD_OK;
  const spd_model_cfg &t = ctx->cfg.target, &d = ctx->cfg.draft;
  const size_t dm = t.d_model > d.d_model ? t.d_model : d.d_model;
  const size_t fm = t.d_ffn > d.d_ffn ? t.d_ffn : d.d_ffn;
  const size_t hm = t.n_heads > d.n_heads ? t.n_heads : d.n_heads;
  const size_t ad = ctx->cfg.draft_adapter_in;
  size_t kin = dm > fm ? dm : fm;
  if (ad > kin) kin = ad;
  const size_t wide = 3 * dm > 2 * fm ? 3 * dm : 2 * fm;
  const size_t rp = ((size_t)R + 63) / 64 * 64;
  spd_status s;   // earlier buffers stay in the context's allocation list until spd_destroy
  if ((s = dalloc(ctx, &ctx->pf.h_hi, rp * kin))) return s;
  if ((s = dalloc(ctx, &ctx->pf.h_lo, rp * kin))) return s;
  if ((s = dalloc(ctx, &ctx->pf.q_hi, rp * dm))) return s;
  if ((s = dalloc(ctx, &ctx->pf.q_lo, rp * dm))) return s;
  if ((s = dalloc(ctx, &ctx->pf.vT, dm * rp))) return s;
  if ((s = dalloc(ctx, &ctx->pf.wide, rp * wide))) return s;
  if ((s = dalloc(ctx, &ctx->pf.S, hm * rp * rp))) return s;
  if ((s = dalloc(ctx, &ctx->pf.p_hi, hm * rp * rp))) return s;
  if ((s = dalloc(ctx, &ctx->pf.p_lo, hm * rp * rp))) return s;
  if ((s = dalloc(ctx, &ctx->pf.g_hi, rp * fm))) return s;
  if ((s = dalloc(ctx, &ctx->pf.g_lo, rp * fm))) return s;
  ctx->pf.cap_rows = rp;
  return SPD_OK;
}

// Dense forward of rows X [R][d] (fp32, device; positions 0..R-1) through every layer of a
// bf16 model: fills the KV cache rows 0..R-1 and leaves the final residual stream in X.
spd_status prefill_tc(spd_ctx* ctx, ModelHost& mh, float* X, int R) {
  const int d = mh.cfg.d_model, f = mh.cfg.d_ffn, H = mh.cfg.n_heads, dh = d / H, L = mh.cfg.n_layers;
  const int rp = (R + 63) / 64 * 64;
  spd_status s;
  if ((s = prefill_scratch(ctx, R))) return s;
  auto& pf = ctx->pf;
  cudaStream_t cs = ctx->stream;
  CU(cudaMemsetAsync(pf.vT, 0, (size_t)d * rp * 2, cs));
  const size_t max_seq = ctx->cfg.max_seq;
  for (int l = 0; l < L; ++l) {
    const ModelHost::RowMajor& w = mh.rm[l];
    __nv_bfloat16* kc = static_cast<__nv_bfloat16*>(mh.md.kcache) + (size_t)l * max_seq * d;
    __nv_bfloat16* vc = static_cast<__nv_bfloat16*>(mh.md.vcache) + (size_t)l * max_seq * d;
    TcArgs a{};
    // attention block
    rms_split_kernel<<<R, 256, 0, cs>>>(X, w.attn_norm, mh.cfg.rms_eps, d, pf.h_hi, pf.h_lo);
    a = TcArgs{}; a.M = R; a.N = 3 * d; a.K = d; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = pf.wide; a.ldo = 3 * d;
    if ((s = tc_gemm(ctx, {pf.h_hi, d, R, 1, (size_t)d * 2, (size_t)R * d * 2}, {pf.h_lo, d, R, 1, (size_t)d * 2, (size_t)R * d * 2},
                     {w.wqkv, d, 3 * d, 1, (size_t)d * 2, (size_t)3 * d * d * 2}, a))) return s;
    rope_kv_kernel<<<592, 256, 0, cs>>>(pf.wide, R, d, dh, 0, mh.md.rope_cos, mh.md.rope_sin, pf.q_hi, pf.q_lo, kc, vc,
                                        pf.vT, rp, (int)max_seq);
    a = TcArgs{}; a.M = R; a.N = R; a.K = dh; a.mode = TC_OUT_F32; a.alpha = mh.md.scale; a.out_f32 = pf.S; a.ldo = rp;
    a.out_batch = (long long)R * rp;
    if ((s = tc_gemm(ctx, {pf.q_hi, dh, R, H, (size_t)d * 2, (size_t)dh * 2}, {pf.q_lo, dh, R, H, (size_t)d * 2, (size_t)dh * 2},
                     {kc, dh, R, H, (size_t)dh * 2, max_seq * dh * 2}, a))) return s;   // a head's cached rows are contiguous
    softmax_causal_split_kernel<<<H * R, 256, 0, cs>>>(pf.S, R, rp, pf.p_hi, pf.p_lo);
    a = TcArgs{}; a.M = R; a.N = dh; a.K = rp; a.mode = TC_OUT_SPLIT; a.alpha = 1.f; a.out_hi = pf.h_hi; a.out_lo = pf.h_lo;
    a.ldo = d; a.out_batch = dh;
    if ((s = tc_gemm(ctx, {pf.p_hi, rp, R, H, (size_t)rp * 2, (size_t)R * rp * 2}, {pf.p_lo, rp, R, H, (size_t)rp * 2, (size_t)R * rp * 2},
                     {pf.vT, rp, dh, H, (size_t)rp * 2, (size_t)dh * rp * 2}, a))) return s;
    a = TcArgs{}; a.M = R; a.N = d; a.K = d; a.mode = TC_OUT_F32_ADD; a.alpha = 1.f; a.out_f32 = X; a.ldo = d;
    if ((s = tc_gemm(ctx, {pf.h_hi, d, R, 1, (size_t)d * 2, (size_t)R * d * 2}, {pf.h_lo, d, R, 1, (size_t)d * 2, (size_t)R * d * 2},
                     {w.wo, d, d, 1, (size_t)d * 2, (size_t)d * d * 2}, a))) return s;
    // feed-forward block
    rms_split_kernel<<<R, 256, 0, cs>>>(X, w.ffn_norm, mh.cfg.rms_eps, d, pf.h_hi, pf.h_lo);
    // gate/up with SwiGLU in the epilogue (interleaved gate/up rows): hi/lo [R][f] straight out of the GEMM
    a = TcArgs{}; a.M = R; a.N = 2 * f; a.K = d; a.mode = TC_OUT_SWIGLU; a.alpha = 1.f; a.out_hi = pf.g_hi; a.out_lo = pf.g_lo; a.ldo = f;
    if ((s = tc_gemm(ctx, {pf.h_hi, d, R, 1, (size_t)d * 2, (size_t)R * d * 2}, {pf.h_lo, d, R, 1, (size_t)d * 2, (size_t)R * d * 2},
                     {w.wgu, d, 2 * f, 1, (size_t)d * 2, (size_t)2 * f * d * 2}, a))) return s;
    a = TcArgs{}; a.M = R; a.N = d; a.K = f; a.mode = TC_OUT_F32_ADD; a.alpha = 1.f; a.out_f32 = X; a.ldo = d;
    if ((s = tc_gemm(ctx, {pf.g_hi, f, R, 1, (size_t)f * 2, (size_t)R * f * 2}, {pf.g_lo, f, R, 1, (size_t)f * 2, (size_t)R * f * 2},
                     {w.wd, f, d, 1, (size_t)f * 2, (size_t)d * f * 2}, a))) return s;
    CU(cudaGetLastError());
  }
  return SPD_OK;
}

// Buffers of a context that are not part of a model: device state, barrier pool, uniforms,
// draft distributions, prefill staging, output ids, pinned state copy, events, graph stream.
spd_status alloc_ctx_buffers(spd_ctx* ctx) {
  const spd_cfg* cfg = &ctx->cfg;
  const int V = cfg->target.vocab;
  const int dmax = cfg->target.d_model > cfg->draft.d_model ? cfg->target.d_model : cfg->draft.d_model;
  spd_status s;
  if ((s = dalloc(ctx, &ctx->st, 1))) return s;
  if ((s = dalloc(ctx, &ctx->bars, (size_t)32 * BAR_POOL))) return s;
  if ((s = dalloc(ctx, &ctx->ubuf, 16))) return s;
  if ((s = dalloc(ctx, &ctx->qbuf, (size_t)MAX_M * V))) return s;   // chain: gamma rows; tree: one per block row
  ctx->truncate = !cfg->greedy && ((cfg->top_k >= 1 && cfg->top_k < V) || (cfg->top_p > 0.f && cfg->top_p < 1.f));
  if (ctx->truncate) {
    if ((s = dalloc(ctx, &ctx->prow, (size_t)MAX_M * V))) return s;
    // one CTA holds a whole row in shared memory
    if ((size_t)V * sizeof(float) + sizeof(TruncScratch) + 1024 > (size_t)ctx->smem_optin)
      return fail(ctx, SPD_EINVAL, "top-k / top-p: a vocabulary row does not fit the shared memory of one CTA");
    if (cudaFuncSetAttribute((const void*)truncate_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)((size_t)V * sizeof(float))) != cudaSuccess)
      return fail(ctx, SPD_ECUDA, "cannot size the truncation kernel's shared memory");
  }
  if ((s = dalloc(ctx, &ctx->rows, (size_t)cfg->max_seq * dmax))) return s;
  if ((s = dalloc(ctx, &ctx->ids_dev, (size_t)cfg->max_seq))) return s;
  ctx->out_cap = cfg->max_seq + MAX_M;
  if ((s = dalloc(ctx, &ctx->out_dev, (size_t)ctx->out_cap))) return s;
  if (cudaMallocHost(&ctx->st_host, sizeof(DevState)) != cudaSuccess) return fail(ctx, SPD_ENOMEM, "pinned allocation failed");
  for (auto& e : ctx->ev)
    if (cudaEventCreate(&e) != cudaSuccess) return fail(ctx, SPD_ECUDA, "event creation failed");
  if (cudaStreamCreateWithFlags(&ctx->gs, cudaStreamNonBlocking) != cudaSuccess)
    return fail(ctx, SPD_ECUDA, "stream creation failed");
  return SPD_OK;
}

// bf16 models take the dense tensor-core prefill; fp32 models go through the M <= 8 kernel in
// chunks of 8 rows.
bool use_tc_prefill(const ModelHost& mh) { return mh.cfg.dtype == 1; }

}  // namespace

// ------------------------------------------------------------------------------ fixed scratch
// Scratch of spd_skinny_gemm_noalloc: lives in the library image, so no allocation call is
// ever made for it.  Layout: [0,256) grid-barrier word, [256,512) kernel status block,
// [512, ...) the streaming-layout copy of the weight matrix.
constexpr size_t NOALLOC_HEADER = 512;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_HEADER + SPD_NOALLOC_MAX_PACKED_BYTES];

// ------------------------------------------------------------------------------ C ABI

extern "C" {

const char* spd_last_error(const spd_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

static void destroy_now(spd_ctx* ctx) {
  cudaStreamSynchronize(ctx->stream);
  if (ctx->gs) cudaStreamSynchronize(ctx->gs);
  if (ctx->block_exec) cudaGraphExecDestroy(ctx->block_exec);
  if (ctx->gs) cudaStreamDestroy(ctx->gs);
  for (void* p : ctx->allocs) cudaFree(p);
  if (ctx->st_host) cudaFreeHost(ctx->st_host);
  for (auto& e : ctx->ev)
    if (e) cudaEventDestroy(e);
  delete ctx;
}

void spd_destroy(spd_ctx* ctx) {
  if (!ctx) return;
  if (ctx->n_forks > 0) {   // forks still read this context's weights: free it with the last of them
    cudaStreamSynchronize(ctx->stream);
    ctx->zombie = true;
    return;
  }
  spd_ctx* origin = ctx->origin;
  destroy_now(ctx);
  if (origin && --origin->n_forks == 0 && origin->zombie) destroy_now(origin);
}

spd_status spd_fork(spd_ctx* parent, spd_ctx** out) {
  if (out) *out = nullptr;
  if (!parent || !out) return SPD_EINVAL;
  if (parent->zombie) return fail(parent, SPD_ESTATE, "spd_fork on a destroyed context");
  spd_ctx* origin = parent->origin ? parent->origin : parent;   // forks of forks hang off the owner of the weights
  spd_ctx* ctx = new (std::nothrow) spd_ctx();
  if (!ctx) return SPD_ENOMEM;
  ctx->cfg = parent->cfg;
  ctx->stream = parent->stream;
  ctx->device = parent->device; ctx->n_sm = parent->n_sm; ctx->smem_optin = parent->smem_optin;
  ctx->target = origin->target;     // copies the descriptors: weight pointers are shared ...
  ctx->draft = origin->draft;
  ctx->target.pos_base = 0; ctx->draft.pos_base = 0;
  spd_status s = alloc_sequence_state(ctx, ctx->target);   // ... the per-sequence buffers are new
  if (!s) s = alloc_sequence_state(ctx, ctx->draft);
  if (!s) s = alloc_ctx_buffers(ctx);
  if (!s && cudaStreamSynchronize(ctx->stream) != cudaSuccess) s = fail(ctx, SPD_ECUDA, "sync failed");
  if (s) {
    parent->err = "spd_fork: " + ctx->err;
    destroy_now(ctx);
    return s;
  }
  ctx->origin = origin;
  origin->n_forks++;
  *out = ctx;
  return SPD_OK;
}

spd_status spd_create(const spd_weights* target_w, const spd_weights* draft_w, const spd_cfg* cfg, spd_ctx** out) {
  if (out) *out = nullptr;
  if (!target_w || !draft_w || !cfg || !out) return SPD_EINVAL;
  spd_ctx* ctx = new (std::nothrow) spd_ctx();
  if (!ctx) return SPD_ENOMEM;
  auto bail = [&](spd_status s) {
    fprintf(stderr, "spd_create: %s\n", ctx->err.c_str());
    spd_destroy(ctx);
    return s;
  };
  ctx->cfg = *cfg;
  ctx->stream = static_cast<cudaStream_t>(cfg->stream);
  spd_status s;
  if ((s = check_model(ctx, cfg->target, "target"))) return bail(s);
  if ((s = check_model(ctx, cfg->draft, "draft"))) return bail(s);
  if (cfg->target.vocab != cfg->draft.vocab) return bail(fail(ctx, SPD_EINVAL, "target and draft vocab differ"));
  if (cfg->gamma_max < 0 || cfg->gamma_max > MAX_M - 1) return bail(fail(ctx, SPD_EINVAL, "gamma_max must be 0..7"));
  if (cfg->max_seq < 16) return bail(fail(ctx, SPD_EINVAL, "max_seq too small"));
  if (!cfg->greedy && !(cfg->temperature > 0.f)) return bail(fail(ctx, SPD_EINVAL, "temperature must be > 0"));
  if (cfg->draft_adapter_in < 0 || cfg->draft_adapter_in % 8) return bail(fail(ctx, SPD_EINVAL, "bad draft_adapter_in"));
  if (cfg->top_k < 0 || !(cfg->top_p >= 0.f)) return bail(fail(ctx, SPD_EINVAL, "top_k and top_p must not be negative"));
  if (cudaGetDevice(&ctx->device) != cudaSuccess) return bail(fail(ctx, SPD_ECUDA, "no CUDA device"));
  cudaDeviceProp prop{};
  if (cudaGetDeviceProperties(&prop, ctx->device) != cudaSuccess) return bail(fail(ctx, SPD_ECUDA, "no device properties"));
  if (prop.major != 10) return bail(fail(ctx, SPD_ECUDA, "this library is built for sm_100a only"));
  if (!prop.cooperativeLaunch) return bail(fail(ctx, SPD_ECUDA, "cooperative launch not supported"));
  ctx->n_sm = prop.multiProcessorCount;
  if (ctx->n_sm > 256) return bail(fail(ctx, SPD_ECUDA, "more than 256 SMs: the per-CTA partial sums are read 8 per lane"));
  ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
  if (cfg->temperature <= 0.f) ctx->cfg.temperature = 1.0f;
  const size_t esz_t = cfg->target.dtype ? 2 : 4, esz_d = cfg->draft.dtype ? 2 : 4;
  size_t stage_elems = 0;
  for (const spd_model_cfg* c : {&cfg->target, &cfg->draft}) {
    const size_t e = c->dtype ? 2 : 4;
    const size_t big = (size_t)(c->vocab > c->d_ffn ? c->vocab : c->d_ffn) * c->d_model * e;
    if (big > stage_elems) stage_elems = big;
  }
  (void)esz_t; (void)esz_d;
  char *staging = nullptr, *rowmajor = nullptr;
  if (cudaMalloc(&staging, stage_elems + 256) != cudaSuccess ||
      cudaMalloc(&rowmajor, 3 * stage_elems + 256) != cudaSuccess) {
    cudaFree(staging);
    return bail(fail(ctx, SPD_ENOMEM, "staging allocation failed"));
  }
  // Launch shape per model.  Default: one CTA per SM, barrier in global memory.  grid_mode 2 runs a
  // model as ONE thread-block cluster (16 CTAs, else 8) whose members synchronise through each
  // other's shared memory: barriers cost a hop between SMs instead of two trips to L2, but 16 SMs'
  // compute warps consume a weight stage every 0.3 us each, far less than 148 do, and the 115M
  // draft's step took 0.61 ms that way against 0.31 ms on the full grid -- so it is not chosen
  // automatically.  The weights are packed for the CTA count of the model.
  for (ModelHost* mh : {&ctx->target, &ctx->draft}) {
    const spd_model_cfg& c = mh == &ctx->target ? cfg->target : cfg->draft;
    mh->grid = ctx->n_sm; mh->cluster = 0;
    const double bytes = ((double)c.n_layers * (4.0 * c.d_model * c.d_model + 3.0 * c.d_model * c.d_ffn) +
                          (double)c.vocab * c.d_model) * (c.dtype ? 2 : 4);
    (void)bytes;
    if (cfg->grid_mode != 2) continue;
    for (int cs : {16, 8}) {
      bool ok = true;
      for (int M = 1; M <= MAX_M && ok; ++M) {
        KernelFn fn = pick_kernel(M, c.dtype);
        LaunchCfg lc{};
        ok = launch_cfg(ctx, fn, M, cs, ctx->smem_optin, &lc) == SPD_OK && cluster_fits(fn, cs, lc.smem);
      }
      if (ok) { mh->grid = cs; mh->cluster = cs; break; }
    }
  }
  s = build_model(ctx, ctx->target, cfg->target, target_w, 0, staging, rowmajor);
  if (!s) s = build_model(ctx, ctx->draft, cfg->draft, draft_w, cfg->draft_adapter_in, staging, rowmajor);
  cudaStreamSynchronize(ctx->stream);
  cudaFree(staging);
  cudaFree(rowmajor);
  if (s) return bail(s);
  if ((s = alloc_ctx_buffers(ctx))) return bail(s);
  // every kernel variant that can be launched must fit one CTA per SM
  for (int M = 1; M <= MAX_M; ++M)
    for (int dt : {cfg->target.dtype, cfg->draft.dtype}) {
      KernelFn fn = pick_kernel(M, dt);
      LaunchCfg lc{};
      if ((s = launch_cfg(ctx, fn, M, ctx->n_sm, ctx->smem_optin, &lc))) return bail(s);
      int nb = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, (const void*)fn, ENGINE_THREADS, lc.smem) != cudaSuccess || nb < 1)
        return bail(fail(ctx, SPD_ECUDA, "forward kernel does not fit on an SM"));
    }
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return bail(fail(ctx, SPD_ECUDA, "sync failed"));
  *out = ctx;
  return SPD_OK;
}

spd_status spd_prefill(spd_ctx* ctx, const float* image_embeds, int m, const float* draft_image_feats,
                       const int32_t* prompt_ids, int n, const float* u0, int32_t* first_token) {
  if (!ctx) return SPD_EINVAL;
  if (n < 1 || m < 0 || !prompt_ids || (m > 0 && !image_embeds)) return fail(ctx, SPD_EINVAL, "bad prefill arguments");
  if (!ctx->cfg.greedy && !u0) return fail(ctx, SPD_EINVAL, "u0 required when sampling");
  const int ad = ctx->cfg.draft_adapter_in;
  if (ad > 0 && (m == 0 || !draft_image_feats)) return fail(ctx, SPD_EINVAL, "draft adapter needs image features");
  if (m + n + ctx->cfg.gamma_max + 1 > ctx->cfg.max_seq) return fail(ctx, SPD_EOVERFLOW, "prompt does not fit max_seq");
  const int V = ctx->cfg.target.vocab;
  std::vector<int32_t> ids_h;
  if (!is_device_ptr(prompt_ids)) {
    for (int i = 0; i < n; ++i)
      if (prompt_ids[i] < 0 || prompt_ids[i] >= V) return fail(ctx, SPD_EINVAL, "prompt id out of range");
  }
  CU(cudaMemcpyAsync(ctx->ids_dev, prompt_ids, n * sizeof(int32_t), cudaMemcpyDefault, ctx->stream));
  int32_t last_id = 0;
  CU(cudaMemcpyAsync(&last_id, ctx->ids_dev + n - 1, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
  float u = u0 ? *u0 : 0.f;
  if (u < 0.f || u >= 1.f) return fail(ctx, SPD_EINVAL, "uniform outside [0,1)");
  CU(cudaMemcpyAsync(ctx->ubuf + 8, &u, sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemsetAsync(ctx->st, 0, sizeof(DevState), ctx->stream));
  CU(cudaMemcpyAsync(&ctx->st->out_cap, &ctx->out_cap, sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  spd_status s;
  ModelHost& dm = ctx->draft;
  ModelHost& tm = ctx->target;
  bool moved_logits = false;
  if (use_tc_prefill(dm) && use_tc_prefill(tm)) {
    // ---- dense tensor-core pass over all rows of each model
    const int dd = dm.cfg.d_model, dt = tm.cfg.d_model;
    const int Rd = (ad > 0 ? m : 0) + n, Rt = m + n;
    if ((s = prefill_scratch(ctx, Rt > Rd ? Rt : Rd))) return s;
    float* X = ctx->rows;
    dm.pos_base = 0;
    if (ad > 0 && dm.rows_given) {   // draft rows [given image rows ; embed(prompt)]
      CU(cudaMemcpyAsync(X, draft_image_feats, (size_t)m * dd * sizeof(float), cudaMemcpyDefault, ctx->stream));
      dm.pos_base = m;
    } else if (ad > 0) {   // draft rows [H W_a^T ; embed(prompt)]
      CU(cudaMemcpyAsync(ctx->pf.wide, draft_image_feats, (size_t)m * ad * sizeof(float), cudaMemcpyDefault, ctx->stream));
      split_rows_kernel<<<592, 256, 0, ctx->stream>>>(ctx->pf.wide, ctx->pf.h_hi, ctx->pf.h_lo, (size_t)m * ad);
      TcArgs a{}; a.M = m; a.N = dd; a.K = ad; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = X; a.ldo = dd;
      if ((s = tc_gemm(ctx, {ctx->pf.h_hi, ad, m, 1, (size_t)ad * 2, (size_t)m * ad * 2},
                       {ctx->pf.h_lo, ad, m, 1, (size_t)ad * 2, (size_t)m * ad * 2},
                       {dm.adapter_rm, ad, dd, 1, (size_t)ad * 2, (size_t)dd * ad * 2}, a))) return s;
      dm.pos_base = m;
    }
    gather_rows_kernel<<<592, 256, 0, ctx->stream>>>(ctx->ids_dev, dm.md.embed, X + (size_t)dm.pos_base * dd, n, dd, V,
                                                       &ctx->st->err);
    if ((s = prefill_tc(ctx, dm, X, Rd))) return s;
    // ---- target rows [V_1..V_m ; embed(prompt)] (Eq. 1); last row -> first generated token
    tm.pos_base = m;
    if (m > 0)
      CU(cudaMemcpyAsync(X, image_embeds, (size_t)m * dt * sizeof(float), cudaMemcpyDefault, ctx->stream));
    gather_rows_kernel<<<592, 256, 0, ctx->stream>>>(ctx->ids_dev, tm.md.embed, X + (size_t)m * dt, n, dt, V, &ctx->st->err);
    if ((s = prefill_tc(ctx, tm, X, Rt))) return s;
    CU(cudaMemcpyAsync(tm.md.x, X + (size_t)(Rt - 1) * dt, dt * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
    StepArgs a = base_args(ctx, tm);
    a.mode = MODE_ROWS; a.skip_layers = 1; a.want_sample = 1;
    a.stat_r0 = 0; a.stat_n = 1;
    a.rows = tm.md.x; a.rows_pos0 = Rt - 1;
    a.init_n_text = n; a.init_prev = last_id;
    a.uniforms = ctx->ubuf + 8; a.out_ids = ctx->out_dev;
    if ((s = launch_model(ctx, tm, 1, a, ctx->stream))) return s;
    moved_logits = true;
  } else {
  // ---- draft: [adapter(features) ; embed(prompt)] or embed(prompt) alone (Sec. 3)
  dm.pos_base = 0;
  if (ad > 0) {
    const int dd = dm.cfg.d_model;
    float* outrows = ctx->rows;
    // stage features at the end of the rows buffer so that outputs can start at 0
    float* fstage = ctx->rows + (size_t)ctx->cfg.max_seq * (ctx->target.cfg.d_model > dd ? ctx->target.cfg.d_model : dd) - (size_t)m * ad;
    if ((size_t)m * ad + (size_t)m * dd > (size_t)ctx->cfg.max_seq * (ctx->target.cfg.d_model > dd ? ctx->target.cfg.d_model : dd))
      return fail(ctx, SPD_EOVERFLOW, "image features do not fit the staging buffer");
    CU(cudaMemcpyAsync(dm.rows_given ? outrows : fstage, draft_image_feats, (size_t)m * ad * sizeof(float),
                       cudaMemcpyDefault, ctx->stream));
    for (int r = 0; r < m && !dm.rows_given; r += MAX_M) {
      const int M = (m - r) < MAX_M ? (m - r) : MAX_M;
      StepArgs a = base_args(ctx, dm);
      a.mode = MODE_GEMM;
      a.gx = fstage + (size_t)r * ad; a.gw = dm.adapter; a.gy = outrows + (size_t)r * dd; a.gN = dd; a.gK = ad;
      if ((s = launch_model(ctx, dm, M, a, ctx->stream))) return s;
    }
    if ((s = feed_rows(ctx, dm, outrows, nullptr, 0, m, 0, false, 0, 0))) return s;
    dm.pos_base = m;
  }
  if ((s = feed_rows(ctx, dm, nullptr, ctx->ids_dev, 0, n, dm.pos_base, false, 0, 0))) return s;
  // ---- target: [V_1..V_m ; embed(prompt)] (Eq. 1); last row -> first generated token
  tm.pos_base = m;
  if (m > 0) {
    CU(cudaMemcpyAsync(ctx->rows, image_embeds, (size_t)m * tm.cfg.d_model * sizeof(float), cudaMemcpyDefault, ctx->stream));
    if ((s = feed_rows(ctx, tm, ctx->rows, nullptr, 0, m, 0, false, 0, 0))) return s;
  }
  if ((s = feed_rows(ctx, tm, nullptr, ctx->ids_dev, 0, n, m, true, n, last_id))) return s;
  }
  ctx->prefilled = false;   // until the device has reported no error below
  ctx->drafted_gamma = -1;
  ctx->n_prompt = n; ctx->m_image = m;
  ctx->last_verify_rows = 1; ctx->last_draft_rows = 0;
  // the sampled row was row (chunk rows - 1) of the last chunk: move it to row 0
  if (!moved_logits) {
    const int lastM = (n % MAX_M) ? (n % MAX_M) : MAX_M;
    if (lastM > 1)
      CU(cudaMemcpyAsync(tm.logits, tm.logits + (size_t)(lastM - 1) * V, V * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
  }
  if ((s = sync_state(ctx))) return s;
  ctx->prefilled = true;
  if (first_token) *first_token = ctx->st_host->pending;
  return SPD_OK;
}

spd_status spd_image_adapter(spd_ctx* ctx, const float* feats, int m, int d_in, const void* w1, int d_hid,
                             const void* w2, int d_out, float* out) {
  if (!ctx) return SPD_EINVAL;
  if (!feats || !w1 || !w2 || !out || m < 1 || d_in < 8 || d_hid < 8 || d_out < 1 || d_in % 8 || d_hid % 8)
    return fail(ctx, SPD_EINVAL, "bad image adapter arguments (widths must be multiples of 8)");
  if (!is_device_ptr(w1) || !is_device_ptr(w2) || !is_device_ptr(out))
    return fail(ctx, SPD_EINVAL, "adapter weights and output must be device memory");
  if ((reinterpret_cast<uintptr_t>(w1) | reinterpret_cast<uintptr_t>(w2) | reinterpret_cast<uintptr_t>(out)) & 15)
    return fail(ctx, SPD_EINVAL, "adapter weights and output must be 16-byte aligned");
  spd_status s;
  auto& ia = ctx->ia;
  const size_t n_in = (size_t)m * d_in, n_hid = (size_t)m * d_hid;
  if (n_in > ia.cap_in) {   // earlier buffers stay in the context's allocation list until spd_destroy
    if ((s = dalloc(ctx, &ia.feats, n_in))) return s;
    if ((s = dalloc(ctx, &ia.f_hi, n_in))) return s;
    if ((s = dalloc(ctx, &ia.f_lo, n_in))) return s;
    ia.cap_in = n_in;
  }
  if (n_hid > ia.cap_hid) {
    if ((s = dalloc(ctx, &ia.g_hi, n_hid))) return s;
    if ((s = dalloc(ctx, &ia.g_lo, n_hid))) return s;
    ia.cap_hid = n_hid;
  }
  const float* fdev = feats;
  if (!is_device_ptr(feats)) {
    CU(cudaMemcpyAsync(ia.feats, feats, n_in * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    fdev = ia.feats;
  }
  split_rows_kernel<<<592, 256, 0, ctx->stream>>>(fdev, ia.f_hi, ia.f_lo, n_in);
  // hidden = GELU(H W1^T), kept as a bf16 hi/lo pair (the GELU runs in the GEMM epilogue)
  TcArgs a{}; a.M = m; a.N = d_hid; a.K = d_in; a.mode = TC_OUT_SPLIT; a.alpha = 1.f;
  a.out_hi = ia.g_hi; a.out_lo = ia.g_lo; a.ldo = d_hid;
  if ((s = tc_gemm(ctx, {ia.f_hi, d_in, m, 1, (size_t)d_in * 2, n_in * 2}, {ia.f_lo, d_in, m, 1, (size_t)d_in * 2, n_in * 2},
                   {w1, d_in, d_hid, 1, (size_t)d_in * 2, (size_t)d_hid * d_in * 2}, a, true))) return s;
  // V = hidden W2^T
  a = TcArgs{}; a.M = m; a.N = d_out; a.K = d_hid; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = out; a.ldo = d_out;
  if ((s = tc_gemm(ctx, {ia.g_hi, d_hid, m, 1, (size_t)d_hid * 2, n_hid * 2}, {ia.g_lo, d_hid, m, 1, (size_t)d_hid * 2, n_hid * 2},
                   {w2, d_hid, d_out, 1, (size_t)d_hid * 2, (size_t)d_out * d_hid * 2}, a))) return s;
  // device-side waits are bounded; report one that ran out
  int e = 0;
  CU(cudaMemcpyAsync(&e, &ctx->st->err, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  if (e != DEV_OK) {
    cudaMemsetAsync(&ctx->st->err, 0, sizeof(int), ctx->stream);
    return check_dev_err(ctx, e);
  }
  return SPD_OK;
}

spd_status spd_draft(spd_ctx* ctx, int gamma, const float* uniforms, int32_t* draft_ids, float* draft_probs) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_draft before spd_prefill");
  if (gamma < 1 || gamma > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "gamma out of range");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  if (draft_probs && !is_device_ptr(draft_probs)) return fail(ctx, SPD_EINVAL, "draft_probs must be device memory");
  const int base = ctx->m_image > ctx->draft.pos_base ? ctx->m_image : ctx->draft.pos_base;
  if (base + ctx->len_ub + gamma + 1 > ctx->cfg.max_seq) {
    spd_status s = sync_state(ctx);
    if (s) return s;
    if (base + ctx->len_ub + gamma + 1 > ctx->cfg.max_seq) return fail(ctx, SPD_EOVERFLOW, "KV cache full");
  }
  if (uniforms) CU(cudaMemcpyAsync(ctx->ubuf, uniforms, gamma * sizeof(float), cudaMemcpyDefault, ctx->stream));
  ModelHost& dm = ctx->draft;
  for (int j = 0; j < gamma; ++j) {
    StepArgs a = base_args(ctx, dm);
    a.mode = MODE_DRAFT;
    a.gamma = gamma; a.j = j;
    geom_draft_step(a, j);
    a.uniforms = ctx->ubuf;
    a.q_out = ctx->qbuf;
    a.logits = dm.logits;
    spd_status s = launch_model(ctx, dm, 2, a, ctx->stream);
    if (s) return s;
    // keep this step's logits row (row 1) for spd_get_draft_logits: rows 2.. of the buffer
    if (j + 2 < MAX_M)
      CU(cudaMemcpyAsync(dm.logits + (size_t)(j + 2) * dm.cfg.vocab, dm.logits + (size_t)dm.cfg.vocab,
                         dm.cfg.vocab * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
  }
  ctx->drafted_gamma = gamma;
  ctx->last_draft_rows = gamma < MAX_M - 2 ? gamma : MAX_M - 2;
  bool need_sync = false;
  spd_status s;
  if (draft_probs && !ctx->cfg.greedy)
    CU(cudaMemcpyAsync(draft_probs, ctx->qbuf, (size_t)gamma * dm.cfg.vocab * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
  if ((s = copy_out(ctx, draft_ids, ctx->st->d_ids, gamma * sizeof(int32_t), &need_sync))) return s;
  if (need_sync) CU(cudaStreamSynchronize(ctx->stream));
  return SPD_OK;
}

spd_status spd_verify(spd_ctx* ctx, int gamma, const int32_t* draft_ids, const float* draft_probs,
                      const float* uniforms, int32_t* n_accepted, int32_t* next_token) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_verify before spd_prefill");
  if (gamma < 0 || gamma > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "gamma out of range");
  if (gamma > 0 && ctx->drafted_gamma != gamma && (!draft_ids || (!ctx->cfg.greedy && !draft_probs)))
    return fail(ctx, SPD_ESTATE, "spd_verify needs the ids and probabilities of an spd_draft with the same gamma");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  if (draft_probs && !is_device_ptr(draft_probs)) return fail(ctx, SPD_EINVAL, "draft_probs must be device memory");
  if (ctx->m_image + ctx->len_ub + gamma + 1 > ctx->cfg.max_seq) {
    spd_status s = sync_state(ctx);
    if (s) return s;
    if (ctx->m_image + ctx->len_ub + gamma + 1 > ctx->cfg.max_seq) return fail(ctx, SPD_EOVERFLOW, "KV cache full");
  }
  const int V = ctx->cfg.target.vocab;
  if (draft_ids && gamma > 0) {
    if (!is_device_ptr(draft_ids))
      for (int j = 0; j < gamma; ++j)
        if (draft_ids[j] < 0 || draft_ids[j] >= V) return fail(ctx, SPD_EINVAL, "draft id out of range");
    CU(cudaMemcpyAsync(ctx->st->d_ids, draft_ids, gamma * sizeof(int32_t), cudaMemcpyDefault, ctx->stream));
  }
  if (uniforms) CU(cudaMemcpyAsync(ctx->ubuf + 8, uniforms, (gamma + 1) * sizeof(float), cudaMemcpyDefault, ctx->stream));
  ModelHost& tm = ctx->target;
  StepArgs a = base_args(ctx, tm);
  a.mode = MODE_VERIFY;
  a.gamma = gamma;
  geom_verify_chain(a, gamma);
  a.uniforms = ctx->ubuf + 8;
  a.q_in = draft_probs ? draft_probs : ctx->qbuf;
  a.out_ids = nullptr;
  a.trace = ctx->trace;
  spd_status s = launch_model(ctx, tm, gamma + 1, a, ctx->stream);
  if (s) return s;
  ctx->drafted_gamma = -1;
  ctx->len_ub += gamma + 1;
  ctx->last_verify_rows = gamma + 1;
  bool need_sync = false;
  if ((s = copy_out(ctx, n_accepted, &ctx->st->n_acc, sizeof(int32_t), &need_sync))) return s;
  if ((s = copy_out(ctx, next_token, &ctx->st->next, sizeof(int32_t), &need_sync))) return s;
  if (need_sync) return sync_state(ctx);
  return SPD_OK;
}

// ---- tree blocks

static spd_status tree_scratch(spd_ctx* ctx) {
  if (ctx->tree_cur) return SPD_OK;
  spd_status s;
  const ModelHost &tm = ctx->target, &dm = ctx->draft;
  if ((s = dalloc(ctx, &ctx->tree_stage_t, (size_t)2 * tm.cfg.n_layers * MAX_M * tm.cfg.d_model * tm.esz))) return s;
  if ((s = dalloc(ctx, &ctx->tree_stage_d, (size_t)2 * dm.cfg.n_layers * MAX_M * dm.cfg.d_model * dm.esz))) return s;
  if (!ctx->prow && (s = dalloc(ctx, &ctx->prow, (size_t)MAX_M * ctx->cfg.target.vocab))) return s;
  if ((s = dalloc(ctx, &ctx->tree_cur, (size_t)ctx->cfg.target.vocab))) return s;
  return SPD_OK;
}

static spd_status tree_shape_from_parent(spd_ctx* ctx, int n, const int32_t* parent, TreeShape* sh, unsigned char* sees) {
  if (n < 1 || n > MAX_M - 1 || !parent || parent[0] != -1) return fail(ctx, SPD_EINVAL, "bad tree: 1..7 nodes, parent[0] = -1");
  sh->n = n; sh->depth_max = 0;
  sh->parent[0] = -1; sh->depth[0] = 0; sees[0] = 1;
  for (int i = 1; i <= n; ++i) {
    if (parent[i] < 0 || parent[i] >= i) return fail(ctx, SPD_EINVAL, "bad tree: parent[i] must lie in 0..i-1");
    sh->parent[i] = (signed char)parent[i];
    sh->depth[i] = (signed char)(sh->depth[parent[i]] + 1);
    sees[i] = (unsigned char)(sees[parent[i]] | (1u << i));
    if (sh->depth[i] > sh->depth_max) sh->depth_max = sh->depth[i];
  }
  for (int i = n + 1; i < MAX_M; ++i) { sh->parent[i] = -1; sh->depth[i] = 0; }
  return SPD_OK;
}

// probability rows of the launch's statistic rows (truncated when top-k / top-p is on)
static spd_status tree_prob_rows(spd_ctx* ctx, const StepArgs& a, cudaStream_t stream) {
  prob_rows_kernel<<<ctx->n_sm, SAMPLE_THREADS, 0, stream>>>(a, ctx->prow);
  if (ctx->truncate)
    truncate_rows_kernel<<<a.stat_n, WARP_THREADS, (size_t)a.md.V * sizeof(float), stream>>>(
        ctx->prow, ctx->prow, a.md.V, ctx->cfg.top_k, ctx->cfg.top_p > 0.f ? ctx->cfg.top_p : 1.0f);
  CU(cudaGetLastError());
  return SPD_OK;
}

spd_status spd_draft_tree(spd_ctx* ctx, int depth, const int32_t* branching, const float* uniforms,
                          int32_t* node_ids, int32_t* parent_out, float* draft_probs) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_draft_tree before spd_prefill");
  if (depth < 1 || depth > MAX_M - 1 || !branching) return fail(ctx, SPD_EINVAL, "bad tree depth / branching");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  if (draft_probs && !is_device_ptr(draft_probs)) return fail(ctx, SPD_EINVAL, "draft_probs must be device memory");
  // level-order parent table: every node at depth d-1 gets branching[d-1] children
  int32_t parent[MAX_M + 1];
  int n = 0, lvl_first = 0, lvl_n = 1;
  parent[0] = -1;
  for (int d = 0; d < depth; ++d) {
    if (branching[d] < 1) return fail(ctx, SPD_EINVAL, "branching must be >= 1");
    if ((long long)lvl_n * branching[d] + n > MAX_M - 1 || (long long)lvl_n * branching[d] + n > ctx->cfg.gamma_max)
      return fail(ctx, SPD_EINVAL, "tree has more nodes than gamma_max (at most 7)");
    const int first_new = n + 1;
    for (int k = 0; k < lvl_n; ++k)
      for (int b = 0; b < branching[d]; ++b) parent[++n] = lvl_first + k;
    lvl_first = first_new; lvl_n = n + 1 - first_new;
  }
  TreeShape sh{};
  unsigned char sees[MAX_M];
  spd_status s = tree_shape_from_parent(ctx, n, parent, &sh, sees);
  if (s) return s;
  if ((s = tree_scratch(ctx))) return s;
  const int base = ctx->m_image > ctx->draft.pos_base ? ctx->m_image : ctx->draft.pos_base;
  if (base + ctx->len_ub + n + 1 > ctx->cfg.max_seq) {
    if ((s = sync_state(ctx))) return s;
    if (base + ctx->len_ub + n + 1 > ctx->cfg.max_seq) return fail(ctx, SPD_EOVERFLOW, "KV cache full");
  }
  if (uniforms) CU(cudaMemcpyAsync(ctx->ubuf, uniforms, n * sizeof(float), cudaMemcpyDefault, ctx->stream));
  ModelHost& dm = ctx->draft;
  for (int lev = 0; lev < depth; ++lev) {
    StepArgs a = base_args(ctx, dm);
    a.mode = MODE_DRAFT; a.gamma = n; a.j = lev; a.tree = 1;
    a.uniforms = ctx->ubuf; a.q_out = ctx->qbuf; a.logits = dm.logits;
    int M;
    if (lev == 0) {           // the rows the draft has not seen: [previous token, pending token = root]
      geom_draft_step(a, 0);
      a.geo.slot[1] = 0;      // (already so: the root is block row 0)
      M = 2;
    } else {                  // the nodes of this depth, each attending its ancestors
      M = 0;
      for (int i = 1; i <= n; ++i)
        if (sh.depth[i] == lev) {
          a.geo.slot[M] = (signed char)i; a.geo.depth[M] = (signed char)lev;
          a.geo.sees[M] = sees[i]; a.geo.src[M] = (signed char)(i - 1);
          ++M;
        }
      a.n_slots = n + 1;
      a.stat_r0 = 0; a.stat_n = M;
    }
    if ((s = launch_model(ctx, dm, M, a, ctx->stream))) return s;
    a.fwd_grid = dm.grid; a.sample_r0 = M - 1;
    if (!ctx->cfg.greedy && (s = tree_prob_rows(ctx, a, ctx->stream))) return s;
    tree_draw_kernel<<<1, SAMPLE_THREADS, 0, ctx->stream>>>(a, sh, ctx->prow);
    CU(cudaGetLastError());
  }
  ctx->tree_shape = sh;
  ctx->tree_drafted = true;
  ctx->drafted_gamma = -1;
  bool need_sync = false;
  if (draft_probs && !ctx->cfg.greedy)
    CU(cudaMemcpyAsync(draft_probs, ctx->qbuf, (size_t)(n + 1) * dm.cfg.vocab * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
  if ((s = copy_out(ctx, node_ids, ctx->st->d_ids, n * sizeof(int32_t), &need_sync))) return s;
  if (parent_out) memcpy(parent_out, parent, (n + 1) * sizeof(int32_t));
  if (need_sync) CU(cudaStreamSynchronize(ctx->stream));
  return SPD_OK;
}

spd_status spd_verify_tree(spd_ctx* ctx, int n_nodes, const int32_t* parent, const int32_t* node_ids,
                           const float* draft_probs, const float* uniforms, int32_t* n_accepted, int32_t* path,
                           int32_t* next_token) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_verify_tree before spd_prefill");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  if (draft_probs && !is_device_ptr(draft_probs)) return fail(ctx, SPD_EINVAL, "draft_probs must be device memory");
  if (n_nodes > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "tree has more nodes than gamma_max");
  TreeShape sh{};
  unsigned char sees[MAX_M];
  spd_status s = tree_shape_from_parent(ctx, n_nodes, parent, &sh, sees);
  if (s) return s;
  const int n = n_nodes;
  if ((!node_ids || (!ctx->cfg.greedy && !draft_probs)) &&
      (!ctx->tree_drafted || ctx->tree_shape.n != n || memcmp(ctx->tree_shape.parent, sh.parent, sizeof(sh.parent))))
    return fail(ctx, SPD_ESTATE, "spd_verify_tree needs the ids and probabilities of an spd_draft_tree of the same shape");
  if ((s = tree_scratch(ctx))) return s;
  if (ctx->m_image + ctx->len_ub + n + 1 > ctx->cfg.max_seq) {
    if ((s = sync_state(ctx))) return s;
    if (ctx->m_image + ctx->len_ub + n + 1 > ctx->cfg.max_seq) return fail(ctx, SPD_EOVERFLOW, "KV cache full");
  }
  const int V = ctx->cfg.target.vocab;
  if (node_ids) {
    if (!is_device_ptr(node_ids))
      for (int j = 0; j < n; ++j)
        if (node_ids[j] < 0 || node_ids[j] >= V) return fail(ctx, SPD_EINVAL, "node id out of range");
    CU(cudaMemcpyAsync(ctx->st->d_ids, node_ids, n * sizeof(int32_t), cudaMemcpyDefault, ctx->stream));
  }
  if (uniforms) CU(cudaMemcpyAsync(ctx->ubuf + 8, uniforms, (n + 1) * sizeof(float), cudaMemcpyDefault, ctx->stream));
  ModelHost &tm = ctx->target, &dm = ctx->draft;
  StepArgs a = base_args(ctx, tm);
  a.mode = MODE_VERIFY; a.gamma = n; a.tree = 1;
  for (int i = 0; i <= n; ++i) {
    a.geo.slot[i] = (signed char)i; a.geo.depth[i] = sh.depth[i];
    a.geo.sees[i] = sees[i]; a.geo.src[i] = (signed char)(i - 1);
  }
  a.n_slots = n + 1;
  a.stat_r0 = 0; a.stat_n = n + 1;
  a.uniforms = ctx->ubuf + 8;
  a.q_in = draft_probs ? draft_probs : ctx->qbuf;
  a.out_ids = nullptr;
  if ((s = launch_model(ctx, tm, n + 1, a, ctx->stream))) return s;
  a.fwd_grid = tm.grid; a.sample_r0 = n;
  if (!ctx->cfg.greedy && (s = tree_prob_rows(ctx, a, ctx->stream))) return s;
  tree_verify_kernel<<<1, SAMPLE_THREADS, 0, ctx->stream>>>(a, sh, ctx->prow, ctx->tree_cur);
  // accepted rows move up to the positions they now hold, in both caches (the draft was fed the
  // nodes above the deepest level only)
  for (int pass = 0; pass < 2; ++pass) {
    tree_gather_kernel<<<dim3(MAX_M - 1, tm.cfg.n_layers, 2), 256, 0, ctx->stream>>>(
        ctx->st, tm.md, tm.pos_base, (int)tm.esz, sh.depth_max, ctx->tree_stage_t, pass);
    if (sh.depth_max > 1)
      tree_gather_kernel<<<dim3(MAX_M - 1, dm.cfg.n_layers, 2), 256, 0, ctx->stream>>>(
          ctx->st, dm.md, dm.pos_base, (int)dm.esz, sh.depth_max - 1, ctx->tree_stage_d, pass);
  }
  CU(cudaGetLastError());
  ctx->tree_drafted = false;
  ctx->drafted_gamma = -1;
  ctx->len_ub += sh.depth_max + 1;
  ctx->last_verify_rows = n + 1;
  bool need_sync = false;
  if ((s = copy_out(ctx, n_accepted, &ctx->st->n_acc, sizeof(int32_t), &need_sync))) return s;
  if ((s = copy_out(ctx, next_token, &ctx->st->next, sizeof(int32_t), &need_sync))) return s;
  if ((s = copy_out(ctx, path, ctx->st->path, sh.depth_max * sizeof(int32_t), &need_sync))) return s;
  if (need_sync) return sync_state(ctx);
  return SPD_OK;
}

// ---- several sequences in one pass over the weights

}  // extern "C"

struct spd_batch {
  std::vector<spd_ctx*> seqs;
  spd_ctx* lead = nullptr;      // stream, error word and GEMM scratch of the batch
  int B = 0;
  BatchSeq* seqs_dev = nullptr;
  ModelDev *mds_t = nullptr, *mds_d = nullptr;
  int *rowslot = nullptr, *origins = nullptr, *out_acc = nullptr, *out_next = nullptr;
  float *X = nullptr, *logits = nullptr, *probs = nullptr, *q_all = nullptr, *u_draft = nullptr, *u_verify = nullptr;
  float* gemm_ws = nullptr;     // partial products of K-sliced GEMMs
  int drafted_gamma = -1;
  int last_rows = 0;
  std::vector<void*> allocs;
  // One step (forward + probability rows + sampling / rule kernels) is a fixed sequence of ~10 small
  // launches per layer whose arguments never change (lengths and tokens live on the device), so it
  // is captured once as a CUDA graph per (model, rows per sequence, draft step) and replayed.
  cudaStream_t cap_stream = nullptr;
  struct StepGraph { cudaGraphExec_t exec = nullptr; int seen = 0; };
  StepGraph g_draft[MAX_M][MAX_M];   // [gamma][j]
  StepGraph g_verify[MAX_M + 1];     // [gamma]
  bool graphs_ok = true;
};

namespace {

template <typename T>
spd_status balloc(spd_batch* bt, T** p, size_t n) {
  spd_ctx* ctx = bt->lead;
  void* q = nullptr;
  CU(cudaMalloc(&q, n * sizeof(T) + 256));
  CU(cudaMemsetAsync(q, 0, n * sizeof(T) + 256, ctx->stream));
  bt->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return SPD_OK;
}

constexpr int BATCH_ATTN_SCRATCH = 100 * 1024;   // two CTAs per SM: 16 warps hide each other's dependency stalls
constexpr int BATCH_KSPLIT_MAX = 8;

template <int M>
spd_status launch_batch_attn(spd_ctx* ctx, const ModelDev* mds, const int* origins, int B, int layer, int chain0,
                             int max_split, __nv_bfloat16* o_hi, __nv_bfloat16* o_lo) {
  static bool attr[MAX_DEV];
  const size_t smem = CTRL_BYTES + BATCH_ATTN_SCRATCH;
  if (!attr[ctx->device]) {
    CU(cudaFuncSetAttribute((const void*)batch_attn_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr[ctx->device] = true;
  }
  batch_attn_kernel<M><<<2 * ctx->n_sm, CONSUMER_THREADS, smem, ctx->stream>>>(mds, origins, B, layer, chain0,
                                                                          BATCH_ATTN_SCRATCH, max_split, o_hi, o_lo);
  CU(cudaGetLastError());
  return SPD_OK;
}

spd_status batch_attn(spd_ctx* ctx, int M, const ModelDev* mds, const int* origins, int B, int layer, int chain0,
                      int max_split, __nv_bfloat16* o_hi, __nv_bfloat16* o_lo) {
  switch (M) {
    case 1: return launch_batch_attn<1>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 2: return launch_batch_attn<2>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 3: return launch_batch_attn<3>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 4: return launch_batch_attn<4>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 5: return launch_batch_attn<5>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 6: return launch_batch_attn<6>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    case 7: return launch_batch_attn<7>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
    default: return launch_batch_attn<8>(ctx, mds, origins, B, layer, chain0, max_split, o_hi, o_lo);
  }
}

// Dense forward of the B x M rows of a batched step through every layer and the LM head of one
// model: logits land in bt->logits [B*M][V]; each sequence's K/V rows are appended to its own cache.
spd_status batch_forward(spd_batch* bt, bool draft, int M, int j) {
  spd_ctx* ctx = bt->lead;
  ModelHost& mh = draft ? ctx->draft : ctx->target;
  const int B = bt->B, R = B * M;
  const int d = mh.cfg.d_model, f = mh.cfg.d_ffn, H = mh.cfg.n_heads, dh = d / H, L = mh.cfg.n_layers, V = mh.cfg.vocab;
  spd_status s;
  if ((s = prefill_scratch(ctx, R))) return s;
  auto& pf = ctx->pf;
  cudaStream_t cs = ctx->stream;
  float* X = bt->X;
  const ModelDev* mds = draft ? bt->mds_d : bt->mds_t;
  batch_embed_kernel<<<R, 128, 0, cs>>>(bt->seqs_dev, B, M, draft ? 1 : 0, j, mh.md.embed, d, V, X, bt->rowslot,
                                        bt->origins, &ctx->st->err);
  const Operand h_hi{pf.h_hi, d, R, 1, (size_t)d * 2, (size_t)R * d * 2}, h_lo{pf.h_lo, d, R, 1, (size_t)d * 2, (size_t)R * d * 2};
  // KV splits per head: about two (sequence, head, split) units per SM, never more than a single
  // sequence would use.  (Choosing the split count for an even division of the units over the CTAs
  // was measured slower: 16 x 32 heads in 2 splits balance better than in 1 but pay for the merges,
  // batched verify 12.6 -> 13.3 ms.)
  int attn_split = (2 * ctx->n_sm + B * H - 1) / (B * H);
  if (attn_split > mh.md.nsplit) attn_split = mh.md.nsplit;
  if (attn_split < 1) attn_split = 1;
  // every GEMM here is a few rows against a large weight matrix: cut K so that about one CTA per SM streams
  // K slices: up to one CTA per SM, never a second wave, at least 8 K blocks per slice.  Weight-tile
  // width (256, 160 or 128 rows): a CTA moves (width + 2 x 128) x K / slices bytes per 64 columns of K
  // -- its weight rows plus the hi and lo activation tiles -- so the pair (width, slices) that fits
  // one wave with the fewest bytes per CTA streams fastest; widths whose grid would leave more than
  // half the SMs without a CTA are not considered.
  auto slices = [&](int N, int K, int bn) {
    const int tiles = (N + bn - 1) / bn, kb = (K + TC_BK - 1) / TC_BK;
    int sp = ctx->n_sm / tiles;
    if (sp > BATCH_KSPLIT_MAX) sp = BATCH_KSPLIT_MAX;
    if (sp > kb / 8) sp = kb / 8;
    return sp < 1 ? 1 : sp;
  };
  auto wide = [&](int N, int K) {
    int best = TC_BN;
    double best_cost = 0.0;
    for (int bn : {TC_BN_WIDE, TC_BN_MID, TC_BN}) {
      const int tiles = (N + bn - 1) / bn, sp = slices(N, K, bn);
      if (bn != TC_BN && (tiles * sp * 2 < ctx->n_sm || tiles > ctx->n_sm)) continue;
      const double waves = (double)((tiles * sp + ctx->n_sm - 1) / ctx->n_sm);
      const double cost = waves * (double)(bn + 2 * TC_BM) * K / sp;
      if (best_cost == 0.0 || cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
  };
  auto ksplit = [&](int N, int K) { return slices(N, K, wide(N, K)); };
  // Where a projection is cut into K slices, the kernel that reads its result adds the slices up
  // (in slice order): the rotary / cache-append kernel for QKV, the fused residual + RMSNorm + split
  // kernel for the output and down projections.
  const size_t xs = (size_t)R * d;
  rms_split_kernel<<<R, 256, 0, cs>>>(X, mh.rm[0].attn_norm, mh.cfg.rms_eps, d, pf.h_hi, pf.h_lo);
  for (int l = 0; l < L; ++l) {
    const ModelHost::RowMajor& w = mh.rm[l];
    TcArgs a{};
    a = TcArgs{}; a.M = R; a.N = 3 * d; a.K = d; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = pf.wide; a.ldo = 3 * d;
    const int sq = ksplit(3 * d, d);
    if ((s = tc_gemm(ctx, h_hi, h_lo, {w.wqkv, d, 3 * d, 1, (size_t)d * 2, (size_t)3 * d * d * 2}, a, false, sq, bt->gemm_ws,
                     wide(3 * d, d), true))) return s;
    batch_rope_append_kernel<<<1184, 256, 0, cs>>>(sq > 1 ? bt->gemm_ws : pf.wide, sq, R, M, d, dh, bt->rowslot,
                                                 mh.md.rope_cos, mh.md.rope_sin, mds, l);
    // (the attention kernel leaves its rows as the hi/lo operand of the output projection)
    if ((s = batch_attn(ctx, M, mds, bt->origins, B, l, draft ? j - 1 : 0, attn_split, pf.h_hi, pf.h_lo))) return s;
    a = TcArgs{}; a.M = R; a.N = d; a.K = d; a.mode = TC_OUT_F32_ADD; a.alpha = 1.f; a.out_f32 = X; a.ldo = d;
    const int so = ksplit(d, d);
    if ((s = tc_gemm(ctx, h_hi, h_lo, {w.wo, d, d, 1, (size_t)d * 2, (size_t)d * d * 2}, a, false, so, bt->gemm_ws, wide(d, d),
                     true))) return s;
    resid_rms_split_kernel<<<R, 256, 0, cs>>>(X, bt->gemm_ws, so > 1 ? so : 0, xs, w.ffn_norm, mh.cfg.rms_eps, d, pf.h_hi, pf.h_lo);
    const int sg = ksplit(2 * f, d);
    if (sg == 1) {   // SwiGLU in the GEMM's epilogue
      a = TcArgs{}; a.M = R; a.N = 2 * f; a.K = d; a.mode = TC_OUT_SWIGLU; a.alpha = 1.f; a.out_hi = pf.g_hi; a.out_lo = pf.g_lo; a.ldo = f;
      if ((s = tc_gemm(ctx, h_hi, h_lo, {w.wgu, d, 2 * f, 1, (size_t)d * 2, (size_t)2 * f * d * 2}, a, false, 1, bt->gemm_ws,
                       wide(2 * f, d)))) return s;
    } else {
      a = TcArgs{}; a.M = R; a.N = 2 * f; a.K = d; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = pf.wide; a.ldo = 2 * f;
      if ((s = tc_gemm(ctx, h_hi, h_lo, {w.wgu, d, 2 * f, 1, (size_t)d * 2, (size_t)2 * f * d * 2}, a, false, sg, bt->gemm_ws,
                       wide(2 * f, d)))) return s;
      swiglu_split_kernel<<<296, 256, 0, cs>>>(pf.wide, R, f, pf.g_hi, pf.g_lo);
    }
    a = TcArgs{}; a.M = R; a.N = d; a.K = f; a.mode = TC_OUT_F32_ADD; a.alpha = 1.f; a.out_f32 = X; a.ldo = d;
    const int sd = ksplit(d, f);
    if ((s = tc_gemm(ctx, {pf.g_hi, f, R, 1, (size_t)f * 2, (size_t)R * f * 2}, {pf.g_lo, f, R, 1, (size_t)f * 2, (size_t)R * f * 2},
                     {w.wd, f, d, 1, (size_t)f * 2, (size_t)d * f * 2}, a, false, sd, bt->gemm_ws, wide(d, f), true))) return s;
    // the norm in front of the next layer (or of the LM head) rides on the residual update
    resid_rms_split_kernel<<<R, 256, 0, cs>>>(X, bt->gemm_ws, sd > 1 ? sd : 0, xs,
                                              l + 1 < L ? mh.rm[l + 1].attn_norm : mh.md.final_norm, mh.cfg.rms_eps, d,
                                              pf.h_hi, pf.h_lo);
  }
  TcArgs a{}; a.M = R; a.N = V; a.K = d; a.mode = TC_OUT_F32; a.alpha = 1.f; a.out_f32 = bt->logits; a.ldo = V;
  if ((s = tc_gemm(ctx, h_hi, h_lo, {mh.lm_rm, d, V, 1, (size_t)d * 2, (size_t)V * d * 2}, a, false, ksplit(V, d), bt->gemm_ws, wide(V, d)))) return s;
  CU(cudaGetLastError());
  bt->last_rows = R;
  return SPD_OK;
}

// softmax rows of bt->logits -> bt->probs, truncated when top-k / top-p is on
spd_status batch_probs(spd_batch* bt, int R) {
  spd_ctx* ctx = bt->lead;
  const int V = ctx->cfg.target.vocab;
  batch_softmax_kernel<<<R, SAMPLE_THREADS, 0, ctx->stream>>>(bt->logits, V, ctx->cfg.temperature, bt->probs);
  if (ctx->truncate)
    truncate_rows_kernel<<<R, WARP_THREADS, (size_t)V * sizeof(float), ctx->stream>>>(
        bt->probs, bt->probs, V, ctx->cfg.top_k, ctx->cfg.top_p > 0.f ? ctx->cfg.top_p : 1.0f);
  CU(cudaGetLastError());
  return SPD_OK;
}

spd_status batch_room(spd_batch* bt, int rows, bool draft) {
  for (spd_ctx* c : bt->seqs) {
    const int base = draft ? (c->m_image > c->draft.pos_base ? c->m_image : c->draft.pos_base) : c->m_image;
    if (base + c->len_ub + rows > c->cfg.max_seq) {
      spd_status s = sync_state(c);
      if (s) return s;
      if (base + c->len_ub + rows > c->cfg.max_seq) return fail(bt->lead, SPD_EOVERFLOW, "KV cache of a sequence is full");
    }
  }
  return SPD_OK;
}

// Runs `enqueue` (which issues its launches on ctx->stream) either directly or, from its second use
// on, as a replay of the graph captured from it.  The first use runs eagerly so that one-time set-up
// (scratch growth, kernel attributes) happens outside any capture.
template <class F>
spd_status run_step_graph(spd_batch* bt, spd_batch::StepGraph& g, F enqueue) {
  spd_ctx* ctx = bt->lead;
  if (!bt->graphs_ok || g.seen == 0) { g.seen = 1; return enqueue(); }
  if (!g.exec) {
    if (!bt->cap_stream && cudaStreamCreateWithFlags(&bt->cap_stream, cudaStreamNonBlocking) != cudaSuccess) {
      cudaGetLastError(); bt->graphs_ok = false; return enqueue();
    }
    cudaStream_t user = ctx->stream;
    cudaGraph_t graph = nullptr;
    bool ok = cudaStreamBeginCapture(bt->cap_stream, cudaStreamCaptureModeRelaxed) == cudaSuccess;
    spd_status r = SPD_OK;
    if (ok) {
      ctx->stream = bt->cap_stream;          // the step's launches go to the capturing stream
      r = enqueue();
      ctx->stream = user;
      ok = cudaStreamEndCapture(bt->cap_stream, &graph) == cudaSuccess && r == SPD_OK && graph != nullptr;
    }
    if (ok) ok = cudaGraphInstantiate(&g.exec, graph, 0) == cudaSuccess;
    if (graph) cudaGraphDestroy(graph);
    if (!ok) {                               // capture not available: plain launches from now on
      cudaGetLastError();
      g.exec = nullptr;
      bt->graphs_ok = false;
      return enqueue();
    }
  }
  CU(cudaGraphLaunch(g.exec, ctx->stream));
  return SPD_OK;
}

}  // namespace

extern "C" {

void spd_batch_destroy(spd_batch* bt) {
  if (!bt) return;
  if (bt->lead) cudaStreamSynchronize(bt->lead->stream);
  for (auto& row : bt->g_draft)
    for (auto& g : row)
      if (g.exec) cudaGraphExecDestroy(g.exec);
  for (auto& g : bt->g_verify)
    if (g.exec) cudaGraphExecDestroy(g.exec);
  if (bt->cap_stream) cudaStreamDestroy(bt->cap_stream);
  for (void* p : bt->allocs) cudaFree(p);
  delete bt;
}

spd_status spd_batch_create(spd_ctx* const* seqs, int B, spd_batch** out) {
  if (out) *out = nullptr;
  if (!seqs || !out || B < 1) return SPD_EINVAL;
  spd_ctx* ctx = seqs[0];
  if (!ctx) return SPD_EINVAL;
  const int gm = ctx->cfg.gamma_max > 0 ? ctx->cfg.gamma_max : 1;
  if (B * (gm + 1) > BATCH_ROWS_MAX || B * 2 > BATCH_ROWS_MAX)
    return fail(ctx, SPD_EINVAL, "batch x (gamma_max + 1) rows must fit one 128-row tile");
  if (ctx->cfg.target.dtype != 1 || ctx->cfg.draft.dtype != 1)
    return fail(ctx, SPD_EINVAL, "the batched path needs bf16 models (tensor-core GEMMs)");
  const spd_ctx* origin0 = ctx->origin ? ctx->origin : ctx;
  for (int b = 0; b < B; ++b) {
    spd_ctx* c = seqs[b];
    if (!c) return fail(ctx, SPD_EINVAL, "null sequence in the batch");
    if ((c->origin ? c->origin : c) != origin0 || c->stream != ctx->stream)
      return fail(ctx, SPD_EINVAL, "the sequences of a batch must be forks of one context (shared weights and stream)");
    for (int k = 0; k < b; ++k)
      if (seqs[k] == c) return fail(ctx, SPD_EINVAL, "a sequence appears twice in the batch");
  }
  spd_batch* bt = new (std::nothrow) spd_batch();
  if (!bt) return SPD_ENOMEM;
  bt->lead = ctx; bt->B = B;
  bt->seqs.assign(seqs, seqs + B);
  const int V = ctx->cfg.target.vocab;
  const size_t dmax = ctx->cfg.target.d_model > ctx->cfg.draft.d_model ? ctx->cfg.target.d_model : ctx->cfg.draft.d_model;
  spd_status s = SPD_OK;
  if (!s) s = balloc(bt, &bt->seqs_dev, (size_t)B);
  if (!s) s = balloc(bt, &bt->mds_t, (size_t)B);
  if (!s) s = balloc(bt, &bt->mds_d, (size_t)B);
  if (!s) s = balloc(bt, &bt->rowslot, (size_t)BATCH_ROWS_MAX);
  if (!s) s = balloc(bt, &bt->origins, (size_t)B);
  if (!s) s = balloc(bt, &bt->out_acc, (size_t)B);
  if (!s) s = balloc(bt, &bt->out_next, (size_t)B);
  if (!s) s = balloc(bt, &bt->X, (size_t)BATCH_ROWS_MAX * dmax);
  if (!s) s = balloc(bt, &bt->logits, (size_t)BATCH_ROWS_MAX * V);
  if (!s) s = balloc(bt, &bt->probs, (size_t)BATCH_ROWS_MAX * V);
  if (!s) s = balloc(bt, &bt->q_all, (size_t)B * gm * V);
  if (!s) s = balloc(bt, &bt->u_draft, (size_t)B * MAX_M);
  if (!s) s = balloc(bt, &bt->u_verify, (size_t)B * MAX_M);
  {   // widest split output: [slices][128 rows][max(3 d, 2 f, V)]
    size_t wide = (size_t)V;
    for (const spd_model_cfg* c : {&ctx->cfg.target, &ctx->cfg.draft}) {
      if ((size_t)3 * c->d_model > wide) wide = (size_t)3 * c->d_model;
      if ((size_t)2 * c->d_ffn > wide) wide = (size_t)2 * c->d_ffn;
    }
    if (!s) s = balloc(bt, &bt->gemm_ws, (size_t)BATCH_KSPLIT_MAX * BATCH_ROWS_MAX * wide);
  }
  if (!s && ctx->truncate &&
      cudaFuncSetAttribute((const void*)truncate_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)((size_t)V * sizeof(float))) != cudaSuccess)
    s = fail(ctx, SPD_ECUDA, "cannot size the truncation kernel's shared memory");
  if (s) { spd_batch_destroy(bt); return s; }
  *out = bt;
  return SPD_OK;
}

// (re)reads each sequence's descriptors: a prefill changes the rows in front of the text
static spd_status batch_refresh(spd_batch* bt) {
  spd_ctx* ctx = bt->lead;
  std::vector<BatchSeq> hs(bt->B);
  std::vector<ModelDev> ht(bt->B), hd(bt->B);
  for (int b = 0; b < bt->B; ++b) {
    spd_ctx* c = bt->seqs[b];
    if (!c->prefilled) return fail(ctx, SPD_ESTATE, "a sequence of the batch has not been prefilled");
    hs[b] = BatchSeq{c->st, c->target.pos_base, c->draft.pos_base};
    ht[b] = c->target.md;
    hd[b] = c->draft.md;
  }
  CU(cudaMemcpyAsync(bt->seqs_dev, hs.data(), hs.size() * sizeof(BatchSeq), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(bt->mds_t, ht.data(), ht.size() * sizeof(ModelDev), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaMemcpyAsync(bt->mds_d, hd.data(), hd.size() * sizeof(ModelDev), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));   // the host vectors go out of scope
  return SPD_OK;
}

spd_status spd_batch_draft(spd_batch* bt, int gamma, const float* uniforms, int32_t* draft_ids) {
  if (!bt) return SPD_EINVAL;
  spd_ctx* ctx = bt->lead;
  if (gamma < 1 || gamma > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "gamma out of range");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  spd_status s;
  if ((s = batch_refresh(bt))) return s;
  if ((s = batch_room(bt, gamma + 1, true))) return s;
  const int B = bt->B, V = ctx->cfg.target.vocab;
  if (uniforms) CU(cudaMemcpyAsync(bt->u_draft, uniforms, (size_t)B * gamma * sizeof(float), cudaMemcpyDefault, ctx->stream));
  for (int j = 0; j < gamma; ++j) {
    auto step = [&]() -> spd_status {
      spd_status r;
      if ((r = batch_forward(bt, true, 2, j))) return r;
      if (!ctx->cfg.greedy && (r = batch_probs(bt, 2 * B))) return r;
      batch_draft_sample_kernel<<<B, SAMPLE_THREADS, 0, ctx->stream>>>(
          bt->seqs_dev, ctx->cfg.greedy ? bt->logits : bt->probs, V, gamma, j, ctx->cfg.greedy, bt->u_draft, bt->q_all);
      CU(cudaGetLastError());
      return SPD_OK;
    };
    if ((s = run_step_graph(bt, bt->g_draft[gamma][j], step))) return s;
  }
  bt->last_rows = 2 * B;
  bt->drafted_gamma = gamma;
  for (spd_ctx* c : bt->seqs) { c->drafted_gamma = -1; c->tree_drafted = false; }
  if (draft_ids) {
    const bool host = !is_device_ptr(draft_ids);
    for (int b = 0; b < B; ++b)
      CU(cudaMemcpyAsync(draft_ids + (size_t)b * gamma, bt->seqs[b]->st->d_ids, gamma * sizeof(int32_t), cudaMemcpyDefault, ctx->stream));
    if (host) CU(cudaStreamSynchronize(ctx->stream));
  }
  return SPD_OK;
}

spd_status spd_batch_verify(spd_batch* bt, int gamma, const float* uniforms, int32_t* n_accepted, int32_t* next_token) {
  if (!bt) return SPD_EINVAL;
  spd_ctx* ctx = bt->lead;
  if (gamma < 0 || gamma > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "gamma out of range");
  if (gamma > 0 && bt->drafted_gamma != gamma) return fail(ctx, SPD_ESTATE, "spd_batch_verify needs an spd_batch_draft with the same gamma");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  spd_status s;
  if ((s = batch_refresh(bt))) return s;
  if ((s = batch_room(bt, gamma + 1, false))) return s;
  const int B = bt->B, V = ctx->cfg.target.vocab, M = gamma + 1;
  if (uniforms) CU(cudaMemcpyAsync(bt->u_verify, uniforms, (size_t)B * M * sizeof(float), cudaMemcpyDefault, ctx->stream));
  auto step = [&]() -> spd_status {
    spd_status r;
    if ((r = batch_forward(bt, false, M, 0))) return r;
    if (!ctx->cfg.greedy && (r = batch_probs(bt, B * M))) return r;
    batch_verify_kernel<<<B, SAMPLE_THREADS, 0, ctx->stream>>>(bt->seqs_dev, ctx->cfg.greedy ? bt->logits : bt->probs,
                                                                bt->q_all, ctx->cfg.greedy ? nullptr : bt->u_verify, gamma,
                                                                V, ctx->cfg.greedy, bt->out_acc, bt->out_next);
    CU(cudaGetLastError());
    return SPD_OK;
  };
  if ((s = run_step_graph(bt, bt->g_verify[gamma], step))) return s;
  bt->last_rows = B * M;
  bt->drafted_gamma = -1;
  for (spd_ctx* c : bt->seqs) { c->len_ub += M; c->drafted_gamma = -1; c->last_verify_rows = 0; }
  bool need_sync = false;
  if ((s = copy_out(ctx, n_accepted, bt->out_acc, B * sizeof(int32_t), &need_sync))) return s;
  if ((s = copy_out(ctx, next_token, bt->out_next, B * sizeof(int32_t), &need_sync))) return s;
  if (need_sync) return sync_state(ctx);   // also reports a device-side error (bad id, a wait that ran out)
  return SPD_OK;
}

spd_status spd_batch_get_logits(spd_batch* bt, float* logits, int rows) {
  if (!bt || !logits) return SPD_EINVAL;
  spd_ctx* ctx = bt->lead;
  if (rows < 1 || rows > bt->last_rows) return fail(ctx, SPD_EINVAL, "rows exceed the last batched call");
  CU(cudaMemcpyAsync(logits, bt->logits, (size_t)rows * ctx->cfg.target.vocab * sizeof(float), cudaMemcpyDefault, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return SPD_OK;
}

spd_status spd_batch_verify_bytes(spd_batch* bt, int gamma, double* bytes) {
  if (!bt || !bytes) return SPD_EINVAL;
  spd_ctx* ctx = bt->lead;
  double kv = 0.0;
  for (spd_ctx* c : bt->seqs) {
    spd_status s = sync_state(c);
    if (s) return s;
    const double C = c->m_image + c->st_host->n_text;
    const double kv_row = 2.0 * c->target.cfg.n_layers * c->target.cfg.d_model * c->target.esz;
    kv += kv_row * (C + gamma + 1) + kv_row * (gamma + 1);
  }
  *bytes = (double)ctx->target.wbytes + kv;
  return SPD_OK;
}

spd_status spd_generate(spd_ctx* ctx, int n_new, int gamma, const float* uniforms, int32_t* out_ids,
                        spd_stats* stats) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_generate before spd_prefill");
  if (n_new < 1 || !out_ids) return fail(ctx, SPD_EINVAL, "bad n_new / out_ids");
  if (gamma < 0 || gamma > ctx->cfg.gamma_max) return fail(ctx, SPD_EINVAL, "gamma out of range");
  if (!ctx->cfg.greedy && !uniforms) return fail(ctx, SPD_EINVAL, "uniforms required when sampling");
  if (n_new > ctx->out_cap) return fail(ctx, SPD_EOVERFLOW, "n_new exceeds the output buffer");
  spd_status s = sync_state(ctx);
  if (s) return s;
  {  // the pending token is the first output; uniforms are indexed by block from 0
    int head[2] = {0, 1};   // block, n_emitted
    CU(cudaMemcpyAsync(&ctx->st->block, head, sizeof(head), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(ctx->out_dev, &ctx->st->pending, sizeof(int), cudaMemcpyDeviceToDevice, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    ctx->st_host->n_emitted = 1;
    ctx->st_host->block = 0;
  }
  if (ctx->m_image + ctx->len_ub + n_new + gamma + 1 > ctx->cfg.max_seq)
    return fail(ctx, SPD_EOVERFLOW, "n_new does not fit max_seq");
  const int us = 2 * gamma + 1;
  if (uniforms) {
    const size_t need = (size_t)n_new * us;
    if (need > ctx->upool_cap) {
      if ((s = dalloc(ctx, &ctx->upool, need))) return s;
      ctx->upool_cap = need;
    }
    CU(cudaMemcpyAsync(ctx->upool, uniforms, need * sizeof(float), cudaMemcpyDefault, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));   // the blocks run on the internal stream
  }
  ModelHost &tm = ctx->target, &dm = ctx->draft;
  double ms_d = 0.0, ms_v = 0.0;
  // One block = gamma draft launches + one verify launch.  Everything a block needs (lengths,
  // tokens, block counter, uniforms) lives on the device, so the same CUDA graph is replayed for
  // every block; it is captured once per (gamma, uniform pool) on an internal stream.
  auto enqueue_block = [&](cudaStream_t cs) -> spd_status {
    spd_status r;
    for (int j = 0; j < gamma; ++j) {
      StepArgs a = base_args(ctx, dm);
      a.mode = MODE_DRAFT; a.gamma = gamma; a.j = j;
      geom_draft_step(a, j);
      a.uniforms = uniforms ? ctx->upool : nullptr; a.u_stride = us; a.u_by_block = 1;
      a.q_out = ctx->qbuf; a.logits = dm.logits;
      if ((r = launch_model(ctx, dm, 2, a, cs))) return r;
    }
    StepArgs a = base_args(ctx, tm);
    a.mode = MODE_VERIFY; a.gamma = gamma;
    geom_verify_chain(a, gamma);
    a.uniforms = uniforms ? ctx->upool : nullptr; a.u_stride = us; a.u_by_block = 1;
    a.q_in = ctx->qbuf; a.out_ids = ctx->out_dev;
    return launch_model(ctx, tm, gamma + 1, a, cs);
  };
  const float* pool_key = uniforms ? ctx->upool : nullptr;
  if (ctx->graphs_ok && (!ctx->block_exec || ctx->block_gamma != gamma || ctx->block_upool != pool_key)) {
    if (ctx->block_exec) { cudaGraphExecDestroy(ctx->block_exec); ctx->block_exec = nullptr; }
    cudaGraph_t graph = nullptr;
    bool ok = cudaStreamBeginCapture(ctx->gs, cudaStreamCaptureModeRelaxed) == cudaSuccess;
    if (ok) {
      const spd_status r = enqueue_block(ctx->gs);
      const cudaError_t ce = cudaStreamEndCapture(ctx->gs, &graph);
      ok = r == SPD_OK && ce == cudaSuccess && graph != nullptr;
    }
    if (ok) ok = cudaGraphInstantiate(&ctx->block_exec, graph, 0) == cudaSuccess;
    if (graph) cudaGraphDestroy(graph);
    if (!ok) {   // capture not available here: fall back to plain launches for good
      cudaGetLastError();
      ctx->block_exec = nullptr;
      ctx->graphs_ok = false;
    } else {
      ctx->block_gamma = gamma;
      ctx->block_upool = pool_key;
    }
  }
  CU(cudaEventRecord(ctx->ev[0], ctx->gs));
  int blocks = 0;
  while (ctx->st_host->n_emitted < n_new) {
    if (ctx->block_exec) CU(cudaGraphLaunch(ctx->block_exec, ctx->gs));
    else if ((s = enqueue_block(ctx->gs))) return s;
    if ((s = sync_state(ctx, ctx->gs, true))) return s;
    ms_d += gamma ? (double)(ctx->st_host->t_draft1 - ctx->st_host->t_draft0) * 1e-6 : 0.0;
    ms_v += (double)(ctx->st_host->t_verify1 - ctx->st_host->t_verify0) * 1e-6;
    ++blocks;
    if (blocks > n_new + 1) return fail(ctx, SPD_ECUDA, "block loop made no progress");
  }
  CU(cudaEventRecord(ctx->ev[3], ctx->gs));
  CU(cudaStreamSynchronize(ctx->gs));
  CU(cudaMemcpyAsync(out_ids, ctx->out_dev, n_new * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  ctx->drafted_gamma = -1;
  ctx->last_verify_rows = gamma + 1;
  if (stats) {
    float tot = 0.f;
    cudaEventElapsedTime(&tot, ctx->ev[0], ctx->ev[3]);
    stats->blocks = blocks;
    stats->tokens = n_new;
    const int emitted = ctx->st_host->n_emitted - 1;
    stats->accepted = emitted - blocks;
    stats->tau = blocks ? (float)emitted / blocks : 0.f;
    stats->ms_total = tot; stats->ms_draft = (float)ms_d; stats->ms_verify = (float)ms_v;
    stats->graph_replays = ctx->block_exec ? blocks : 0;
  }
  return SPD_OK;
}

spd_status spd_get_logits(spd_ctx* ctx, float* logits, int rows) {
  if (!ctx || !logits) return SPD_EINVAL;
  if (rows < 1 || rows > ctx->last_verify_rows) return fail(ctx, SPD_EINVAL, "rows exceed the last verify call");
  CU(cudaMemcpyAsync(logits, ctx->target.logits, (size_t)rows * ctx->cfg.target.vocab * sizeof(float), cudaMemcpyDefault, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return SPD_OK;
}

spd_status spd_get_draft_logits(spd_ctx* ctx, float* logits, int rows) {
  if (!ctx || !logits) return SPD_EINVAL;
  if (rows < 1 || rows > ctx->last_draft_rows) return fail(ctx, SPD_EINVAL, "rows exceed the last draft call");
  const int V = ctx->cfg.draft.vocab;
  CU(cudaMemcpyAsync(logits, ctx->draft.logits + (size_t)2 * V, (size_t)rows * V * sizeof(float), cudaMemcpyDefault, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  return SPD_OK;
}

spd_status spd_trace(spd_ctx* ctx, uint64_t* stamps, int cap, int* n) {
  if (!ctx || !n) return SPD_EINVAL;
  const int need = 2 + ctx->cfg.target.n_layers * 18 + 16;
  if (!ctx->trace) {   // first call switches tracing on for later spd_verify calls
    spd_status s = dalloc(ctx, &ctx->trace, (size_t)need);
    if (s) return s;
    ctx->trace_cap = need;
    *n = 0;
    return SPD_OK;
  }
  const int cnt = 1 + ctx->cfg.target.n_layers * 18 + 7;
  *n = cnt < cap ? cnt : cap;
  if (stamps && *n > 0) {
    CU(cudaMemcpyAsync(stamps, ctx->trace, (size_t)*n * sizeof(uint64_t), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
  }
  return SPD_OK;
}

spd_status spd_rollback(spd_ctx* ctx, int n_text, int32_t prev_token, int32_t pending_token) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "spd_rollback before spd_prefill");
  const int V = ctx->cfg.target.vocab;
  if (n_text < 1 || ctx->m_image + n_text + 1 > ctx->cfg.max_seq || prev_token < 0 || prev_token >= V ||
      pending_token < 0 || pending_token >= V)
    return fail(ctx, SPD_EINVAL, "bad rollback arguments");
  int v[3] = {n_text, pending_token, prev_token};
  CU(cudaMemcpyAsync(&ctx->st->n_text, v, sizeof(v), cudaMemcpyHostToDevice, ctx->stream));
  CU(cudaStreamSynchronize(ctx->stream));
  ctx->len_ub = n_text;
  ctx->drafted_gamma = -1;
  return SPD_OK;
}

spd_status spd_get_state(spd_ctx* ctx, int32_t* n_text, int32_t* pending_token) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "no sequence yet");
  spd_status s = sync_state(ctx);
  if (s) return s;
  if (n_text) *n_text = ctx->st_host->n_text;
  if (pending_token) *pending_token = ctx->st_host->pending;
  return SPD_OK;
}

spd_status spd_reject_sample(const float* p, const float* q, const int32_t* ids, const float* u, int B, int gamma,
                             int V, int greedy, int32_t* n_acc, int32_t* next, void* stream) {
  if (!p || !n_acc || !next || B < 1 || gamma < 0 || V < 1) return SPD_EINVAL;
  if (gamma > 0 && !ids) return SPD_EINVAL;
  if (!greedy && (!u || (gamma > 0 && !q))) return SPD_EINVAL;
  reject_sample_kernel<<<B, SAMPLE_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(p, q, ids, u, gamma, V, greedy,
                                                                                    n_acc, next);
  return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ECUDA;
}

spd_status spd_truncate_probs(const float* probs, float* out, int rows, int V, int top_k, float top_p, void* stream) {
  if (!probs || !out || rows < 1 || V < 1 || !(top_p > 0.0f)) return SPD_EINVAL;
  if (!is_device_ptr(probs) || !is_device_ptr(out)) return SPD_EINVAL;
  int dev = 0, optin = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
    return SPD_ECUDA;
  const size_t smem = (size_t)V * sizeof(float);
  if (smem + sizeof(TruncScratch) + 1024 > (size_t)optin) {
    fprintf(stderr, "spd_truncate_probs: a row of %d probabilities does not fit shared memory\n", V);
    return SPD_EINVAL;
  }
  if (cudaFuncSetAttribute((const void*)truncate_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return SPD_ECUDA;
  truncate_rows_kernel<<<rows, WARP_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(probs, out, V, top_k, top_p);
  return cudaGetLastError() == cudaSuccess ? SPD_OK : SPD_ECUDA;
}

// Scratch of the two stand-alone GEMM entry points, per device: a grid-barrier word, a status
// block (DevState: only its error word is used) and, for spd_skinny_gemm, the tile-packed copy of w.
struct GemmScratch {
  bool ready = false;
  unsigned* bar = nullptr;
  DevState* st = nullptr;
  char* packed = nullptr;
  size_t packed_cap = 0;
  int n_sm = 0, smem_optin = 0;
};
static GemmScratch g_gemm_scratch[MAX_DEV];      // spd_skinny_gemm (allocated on first use)
static GemmScratch g_noalloc_state[MAX_DEV];     // spd_skinny_gemm_noalloc (points into g_noalloc_scratch)

spd_status spd_skinny_gemm(const float* x, const void* w, int dtype, int M, int N, int K, float* y, void* stream) {
  if (!x || !w || !y || M < 1 || M > MAX_M || N < 1 || K < 8 || K % 8 || (dtype != 0 && dtype != 1)) return SPD_EINVAL;
  spd_ctx* ctx = nullptr;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return SPD_ECUDA;
  GemmScratch& g = g_gemm_scratch[dev];
  if (!g.ready) {
    cudaDeviceProp prop{};
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SPD_ECUDA;
    if (prop.major != 10) return SPD_ECUDA;
    unsigned* bar = nullptr;
    DevState* st = nullptr;
    if (cudaMalloc(&bar, 256) != cudaSuccess) return SPD_ENOMEM;
    if (cudaMalloc(&st, sizeof(DevState)) != cudaSuccess) { cudaFree(bar); return SPD_ENOMEM; }
    if (cudaMemset(st, 0, sizeof(DevState)) != cudaSuccess) { cudaFree(bar); cudaFree(st); return SPD_ECUDA; }
    g.bar = bar; g.st = st;
    g.n_sm = prop.multiProcessorCount;
    g.smem_optin = (int)prop.sharedMemPerBlockOptin;
    g.ready = true;   // only now: a failed set-up is repeated by the next call
  }
  const size_t esz = dtype == 1 ? 2 : 4;
  const size_t need = packed_bytes(N, K, esz);
  if (need > g.packed_cap) {
    cudaStreamSynchronize(cs);
    if (g.packed) cudaFree(g.packed);
    g.packed = nullptr; g.packed_cap = 0;
    if (cudaMalloc(&g.packed, need) != cudaSuccess) return SPD_ENOMEM;
    g.packed_cap = need;
  }
  spd_status s = pack_tiles(ctx, g.packed, w, N, K, esz, g.n_sm, cs);
  if (s) return s;
  StepArgs a{};
  a.mode = MODE_GEMM;
  a.st = g.st;
  a.gx = x; a.gw = g.packed; a.gy = y; a.gN = N; a.gK = K;
  return launch_forward(ctx, M, dtype, a, cs, g.n_sm, 0, g.smem_optin, g.bar, g.n_sm);
}

spd_status spd_skinny_gemm_status(int noalloc, void* stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return SPD_ECUDA;
  const GemmScratch& g = noalloc ? g_noalloc_state[dev] : g_gemm_scratch[dev];
  if (!g.ready) return SPD_ESTATE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int e = 0;
  if (cudaMemcpyAsync(&e, &g.st->err, sizeof(int), cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaStreamSynchronize(cs) != cudaSuccess)
    return SPD_ECUDA;
  if (e == DEV_OK) return SPD_OK;
  cudaMemsetAsync(&g.st->err, 0, sizeof(int), cs);
  return SPD_ETIMEOUT;
}

spd_status spd_skinny_gemm_noalloc(const float* x, const void* w, int dtype, int M, int N, int K, float* y,
                                   void* stream) {
  if (!x || !w || !y || M < 1 || M > MAX_M || N < 1 || K < 8 || K % 8 || (dtype != 0 && dtype != 1)) return SPD_EINVAL;
  const size_t esz = dtype == 1 ? 2 : 4;
  const size_t need = packed_bytes(N, K, esz);
  if (need > SPD_NOALLOC_MAX_PACKED_BYTES) {
    fprintf(stderr, "spd_skinny_gemm_noalloc: N=%d K=%d needs %zu bytes of scratch, the fixed scratch holds %zu\n", N,
            K, need, (size_t)SPD_NOALLOC_MAX_PACKED_BYTES);
    return SPD_EOVERFLOW;
  }
  // Per-device set-up on the first call with that device current: the array's name is only a
  // host-side handle, the device address comes from the runtime.
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return SPD_ECUDA;
  GemmScratch& g = g_noalloc_state[dev];
  if (!g.ready) {
    cudaDeviceProp prop{};
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess || prop.major != 10) return SPD_ECUDA;
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return SPD_ECUDA;
    g.n_sm = prop.multiProcessorCount;
    g.smem_optin = (int)prop.sharedMemPerBlockOptin;
    g.bar = reinterpret_cast<unsigned*>(ptr);
    g.st = reinterpret_cast<DevState*>(ptr + 256);
    g.packed = reinterpret_cast<char*>(ptr + NOALLOC_HEADER);
    g.packed_cap = SPD_NOALLOC_MAX_PACKED_BYTES;
    g.ready = true;
  }
  spd_ctx* ctx = nullptr;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the last call left: the barrier word and the status block must
  // start at zero (launch_forward clears the barrier word, the status block is cleared here)
  if (cudaMemsetAsync(g.st, 0, 256, cs) != cudaSuccess) return SPD_ECUDA;
  spd_status s = pack_tiles(ctx, g.packed, w, N, K, esz, g.n_sm, cs);
  if (s) return s;
  StepArgs a{};
  a.mode = MODE_GEMM;
  a.st = g.st;
  a.gx = x; a.gw = g.packed; a.gy = y; a.gN = N; a.gK = K;
  return launch_forward(ctx, M, dtype, a, cs, g.n_sm, 0, g.smem_optin, g.bar, g.n_sm);
}

spd_status spd_wait_selftest(spd_ctx* ctx, int which, unsigned polls) {
  if (!ctx) return SPD_EINVAL;
  if ((which != 0 && which != 1) || polls < 1 || polls > (1u << 20)) return fail(ctx, SPD_EINVAL, "bad selftest arguments");
  unsigned* bar = next_bar(ctx);
  CU(cudaMemsetAsync(bar, 0, sizeof(unsigned), ctx->stream));
  wait_selftest_kernel<<<ctx->n_sm, CONSUMER_THREADS, 0, ctx->stream>>>(ctx->st, bar, which, polls);
  CU(cudaGetLastError());
  return sync_state(ctx);   // reads the error word, clears it, maps it to SPD_ETIMEOUT
}

spd_status spd_verify_bytes(spd_ctx* ctx, int gamma, double* bytes) {
  if (!ctx || !bytes) return SPD_EINVAL;
  if (!ctx->prefilled) return fail(ctx, SPD_ESTATE, "no sequence yet");
  spd_status s = sync_state(ctx);
  if (s) return s;
  const ModelHost& tm = ctx->target;
  const double C = ctx->m_image + ctx->st_host->n_text;
  const double kv_row = 2.0 * tm.cfg.n_layers * tm.cfg.d_model * tm.esz;
  *bytes = (double)tm.wbytes + kv_row * (C + gamma + 1) + kv_row * (gamma + 1);
  return SPD_OK;
}

}  // extern "C"
