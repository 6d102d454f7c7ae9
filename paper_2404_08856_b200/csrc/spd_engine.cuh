// The forward engine: ONE persistent cooperative kernel runs a whole M-row forward pass
// (M = gamma+1 rows for the verify step, 2 rows for a draft step, up to 8 rows for a
// chunk of prompt rows) through every layer, the LM head and the sampling rule.
//
// Why one kernel: the step is bound by streaming the weights from HBM once (the paper's
// "memory bandwidth bottleneck", Sec. 1); with a launch per operation the pipeline drains
// at every boundary.  Here a producer warp per CTA streams weight tiles through a ring of
// shared-memory stages with bulk async copies and runs AHEAD of the compute warps across
// layer and phase boundaries (weights never depend on activations), so HBM stays busy
// while the compute warps sit in a grid barrier, build their activation tile or run
// attention.
//
// Per layer (Eq. 1's decoder, LLaMA architecture): RMSNorm -> QKV projection (+ RoPE and
// KV-cache append in the epilogue) | attention of the M new rows over the cache, causal
// within the block | output projection + residual | RMSNorm -> gate/up projection +
// SwiGLU | down projection + residual.  "|" is a grid barrier.
//
// Skinny GEMM Y[M,N] = X[M,K] W[N,K]^T.  Weight rows are dealt to the CTAs in quads (balanced to
// within 4 rows), a CTA's rows are cut into tiles of <= 32 rows and a ring stage is 512 bytes of
// every row of a tile.  The M activation rows sit in shared memory as fp32.
//  * bf16 weights: mma.sync m16n8k16 with the weights as the A operand (ldmatrix from the stage,
//    16-byte chunks swizzled) and the activations as the B operand, split on the fly into two
//    bf16 values (x = hi + lo), fp32 accumulation; the 8 warps split K inside a stage and their
//    partial sums meet once per tile in shared memory.
//  * fp32 weights: warp w owns rows 4w..4w+3 of the tile, lanes split K in 16-byte pieces,
//    packed two-wide fp32 FMAs, butterfly reduction over the lanes.
#pragma once
#include "spd_device.cuh"
#include "spd_sample.cuh"

namespace spd {

constexpr int MAX_M = 8;
constexpr int KC_MAX = 4096;          // activation columns resident in shared memory
constexpr int STAGE_BYTES = 16384;    // 32 rows x 512 B
constexpr int NSTAGE_MAX = 12;
constexpr int CONSUMER_THREADS = 256;
constexpr int ENGINE_THREADS = CONSUMER_THREADS + 32;
constexpr int CTRL_BYTES = 1024;
constexpr int ZERO_BYTES = 512;         // a row of zeros for out-of-range ldmatrix lanes
constexpr int RED_BYTES = 8192;         // cross-warp partial sums of one tile
constexpr int LAYER_SMEM_MAX = 64;       // per-layer pointer records kept in shared memory (more: read from global)
constexpr int LAYER_BYTES = LAYER_SMEM_MAX * 48;
constexpr int PRE_BYTES = 2048;          // epilogue operands fetched asynchronously during a tile's K loop
constexpr int FIXED_SMEM = CTRL_BYTES + ZERO_BYTES + RED_BYTES + LAYER_BYTES + PRE_BYTES;
// activation region: M rows of KC_MAX fp32 (or two bf16 planes), at least 64 KB so that the
// attention phase can stage its K/V tiles there
constexpr int X_PAD = 8;                // floats of padding per activation row (bank spread)
__host__ __device__ constexpr int x_bytes(int M) {
  return M * (KC_MAX + X_PAD) * 4 > 65536 ? M * (KC_MAX + X_PAD) * 4 : 65536;
}

enum : int { MODE_VERIFY = 0, MODE_DRAFT = 1, MODE_ROWS = 2, MODE_GEMM = 3 };
enum : int { PRO_PLAIN = 0, PRO_NORM = 1 };
enum : int { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_QKV = 3 };

struct LayerDev {
  const void *wqkv, *wo, *wgu, *wd;   // repacked: see spd_api.cu
  const float *attn_norm, *ffn_norm;
};
static_assert(sizeof(LayerDev) == 48, "LAYER_BYTES assumes 48-byte records");

struct ModelDev {
  int L, d, H, dh, f, V, max_seq, nsplit;
  float eps, scale;
  const float* embed;                 // token embedding table, fp32 [V][d]
  const void* lm_head;
  const float* final_norm;
  const float *rope_cos, *rope_sin;   // [max_seq][dh/2]
  void *kcache, *vcache;              // [L][H][max_seq][dh]: a head's rows are contiguous (one stream per attention unit)
  float *x, *qbuf, *attn, *act;       // [8][d], [8][d], [8][d], [8][f]
  float *xg;                          // [8][d]: residual stream times the gain of the next RMSNorm
  float *ssq;                         // [grid][8]: per-CTA partial sums of x^2 of the residual stream rows
  float *apart, *aml;                 // attention partials [H][nsplit][8][dh], [H][nsplit][8][2]
  unsigned* head_cnt;                 // [H]
  float* stat_part;                   // [grid][8][4]: row max, row sum, argmax value, argmax index
  unsigned long long* cdf_part;       // [grid][2]: integer mass of the CTA's vocabulary slice, (max weight, index);
                                      // then [2]: accepted count r, (max, sum exp) of row r for the pick kernel
  const LayerDev* layers;
};

struct DevState {
  int n_text;     // committed text tokens, pending excluded = text position of pending
  int pending, prev;
  int block;      // blocks committed since prefill
  int n_emitted;  // tokens written to out_ids
  int err;
  int n_acc, next;
  int d_ids[MAX_M];
  int out_cap;
  int pad[3];
  int path[MAX_M];   // tree blocks: block rows of the accepted nodes, root downwards (n_acc of them)
  // %globaltimer (ns) at the start / end of the last draft steps and verify step
  unsigned long long t_draft0, t_draft1, t_verify0, t_verify1;
};
static_assert(sizeof(DevState) <= 256, "the fixed scratch of spd_skinny_gemm_noalloc reserves 256 bytes for it");

// Geometry of the M rows of a decode launch relative to the ORIGIN = sequence position of the
// pending token (the root of the block).  A plain block is the chain slot = depth = m,
// sees = {0..m}; a token tree (Sec. 5) gives every node its own cache row (slot) while siblings
// share a depth, and a node attends its ancestors and itself only.
struct RowGeom {
  signed char slot[MAX_M];     // K/V cache row = origin + slot (-1: the row of the previous token)
  signed char depth[MAX_M];    // rotary position = origin + depth
  unsigned char sees[MAX_M];   // bit s set: the row attends cache row origin + s; rows below the origin always
  signed char src[MAX_M];      // token of the row: -2 previous token, -1 pending token, k >= 0 draft token k
};

// A token tree below the pending token: block row 0 is the root (the pending token itself), rows
// 1..n are draft nodes in an order in which parents come first.
struct TreeShape {
  int n;                       // draft nodes, 1..MAX_M-1
  int depth_max;               // depth of the deepest node
  signed char parent[MAX_M];   // parent[i] < i: block row of node i's parent; parent[0] = -1
  signed char depth[MAX_M];    // depth[0] = 0
};

struct StepArgs {
  ModelDev md;            // by value: read through the constant bank
  RowGeom geo;
  int n_slots;            // cache rows from the origin on that this launch may attend (max slot + 1)
  int stat_r0, stat_n;    // rows of `logits` whose softmax statistics the kernel leaves for the sampling kernels
  int tree;               // 1: a tree block -- the rule runs in the tree kernels, never inside this kernel
  DevState* st;
  unsigned* bar;          // grid-barrier counter, zero at launch
  int mode, gamma, j, pos_base, nstage, greedy;
  int cluster_ctas;       // > 0: the grid is ONE thread-block cluster of that many CTAs (small models)
  int fwd_grid;           // CTAs of the forward kernel that left the row statistics (set at launch)
  float temperature;
  // MODE_ROWS
  const float* rows;      // fp32 [M, d] input rows (already embeddings), or NULL: ids
  const int* row_ids;     // MODE_ROWS with rows == NULL: token ids [M]
  int rows_pos0, want_sample, init_n_text, init_prev;
  int skip_layers;        // MODE_ROWS: rows are the final residual stream (md.x); run the LM head only
  int sample_r0;          // row of `logits` a draft step / a prefill chunk samples from (set at launch)
  // uniforms
  const float* uniforms;
  int u_stride, u_by_block;
  // draft distributions [gamma][V]
  const float* q_in;
  float* q_out;
  float* logits;          // [M][V] LM-head output
  int* out_ids;
  // MODE_GEMM
  const float* gx; const void* gw; float* gy; int gN, gK;
  // optional phase trace: CTA 0 stores %globaltimer after every phase and every barrier
  unsigned long long* trace;
};

struct Ctrl {
  uint64_t full[NSTAGE_MAX];
  uint64_t empty[NSTAGE_MAX];
  uint64_t xbar;                    // completion of the activation rows' bulk copies
  uint64_t cbar;                    // cluster launches: one arrival per CTA of the cluster per barrier
  SampleScratch sc;
  float red[8][MAX_M];
  float inv[MAX_M];
  float rowmax[MAX_M], rowsum[MAX_M];
  int flag;
  int tok[MAX_M];                   // token ids of the M rows
  int rowslot[MAX_M];               // absolute K/V cache row of each of the M rows
  int rowpos[MAX_M];                // rotary position of each row
  unsigned sees[MAX_M];             // bit s: attends cache row origin + s
  int trace_n;                      // entries written so far (CTA 0 only)
  unsigned long long* trace;        // NULL: tracing off
};

// Trace entry = (%globaltimer ns << 8) | id.  ids: 0 kernel start, 1 activation tile built,
// 2 last weight stage consumed, 3 phase finished, 4 grid barrier passed.
__device__ __forceinline__ void trace_stamp(Ctrl* ctl, int id) {
  if (ctl->trace && threadIdx.x == 0) ctl->trace[ctl->trace_n++] = (globaltimer() << 8) | (unsigned)id;
}
static_assert(sizeof(Ctrl) <= CTRL_BYTES, "control block too large");

struct Gemm {
  const void* W;
  int N, K, pro, epi, layer;
};

__device__ __forceinline__ Gemm get_gemm(const ModelDev& md, const LayerDev* layers, int idx) {
  Gemm g;
  const int l = idx >> 2, which = idx & 3;
  g.layer = l;
  if (l >= md.L) { g.W = md.lm_head; g.N = md.V; g.K = md.d; g.pro = PRO_NORM; g.epi = EPI_STORE; return g; }
  const LayerDev& ly = layers[l];
  switch (which) {
    case 0: g.W = ly.wqkv; g.N = 3 * md.d; g.K = md.d; g.pro = PRO_NORM; g.epi = EPI_QKV; break;
    case 1: g.W = ly.wo; g.N = md.d; g.K = md.d; g.pro = PRO_PLAIN; g.epi = EPI_RESID; break;
    case 2: g.W = ly.wgu; g.N = 2 * md.f; g.K = md.d; g.pro = PRO_NORM; g.epi = EPI_SWIGLU; break;
    default: g.W = ly.wd; g.N = md.d; g.K = md.f; g.pro = PRO_PLAIN; g.epi = EPI_RESID; break;
  }
  return g;
}

template <typename WT> struct WTraits;
template <> struct WTraits<__nv_bfloat16> { static constexpr int EPL = 8; };
template <> struct WTraits<float> { static constexpr int EPL = 4; };

__device__ __forceinline__ void chunking(int K, int kstep, int& nchunk, int& kcl) {
  nchunk = (K + KC_MAX - 1) / KC_MAX;
  kcl = (K + nchunk - 1) / nchunk;
  kcl = (kcl + kstep - 1) / kstep * kstep;
}

// Rows are dealt to CTAs in quads of 4, as evenly as integers allow: CTA c owns quads
// [Q*c/G, Q*(c+1)/G).  Streamed bytes per CTA then differ by at most one quad.
__device__ __forceinline__ void cta_quads(int N, int cta, int G, int& q0, int& q1) {
  const long long Q = (N + 3) >> 2;
  q0 = (int)(Q * cta / G);
  q1 = (int)(Q * (cta + 1) / G);
}

struct Ring {
  int stage;
  unsigned phase;
  int nstage;
  __device__ __forceinline__ void advance() {
    if (++stage == nstage) { stage = 0; phase ^= 1u; }
  }
};

// ------------------------------------------------------------------------------ producer

// Packed weight layout (built once at set-up): the rows of a CTA are contiguous; they are
// cut into tiles of up to 32 rows; a tile is stored step by step, one step = 512 bytes of
// every row of the tile ([row][512 B], so a step of an nr-row tile is one contiguous block
// of nr*512 bytes = one bulk copy = one ring stage).  For bf16 the 16-byte chunks of a row
// are XOR-swizzled with (row & 7) so that ldmatrix reads are bank-conflict free.
template <typename WT>
__device__ void produce_gemm(const Gemm& g, int cta, int G, Ring& ring, Ctrl* ctl, char* stages, uint64_t pol,
                             volatile int* err) {
  constexpr int EPL = WTraits<WT>::EPL, KSTEP = 32 * EPL;
  const int lane = threadIdx.x & 31;
  int q0, q1;
  cta_quads(g.N, cta, G, q0, q1);
  const int rows = (q1 - q0) * 4;
  const int nsteps = (g.K + KSTEP - 1) / KSTEP;
  for (int t = 0; t * 32 < rows; ++t) {
    const int nr = min(32, rows - t * 32);
    const char* src = static_cast<const char*>(g.W) + ((size_t)(q0 * 4 + t * 32) * nsteps) * 512;
    const unsigned bytes = nr * 512;
    for (int s = 0; s < nsteps; ++s) {
      if (!mbar_wait(&ctl->empty[ring.stage], ring.phase ^ 1u, err, DEV_TIMEOUT_EMPTY)) return;
      if (lane == 0) {
        mbar_arrive_expect_tx(&ctl->full[ring.stage], bytes);
        bulk_g2s(stages + (size_t)ring.stage * STAGE_BYTES, src + (size_t)s * bytes, bytes, &ctl->full[ring.stage],
                 pol);
      }
      ring.advance();
    }
  }
}

// KV splits actually used for a context of `len` rows: short contexts are not cut up (a head
// is then finished by one CTA and needs no merge), long ones use up to md.nsplit CTAs per head.
__device__ __forceinline__ int eff_nsplit(const ModelDev& md, int len) {
  const int want = (len + 175) / 176;
  return want < 1 ? 1 : (want < md.nsplit ? want : md.nsplit);
}

// ------------------------------------------------------------------------------ X tile

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Source rows of an activation tile (fp32, 16-byte aligned): row m starts at
// base + (idx ? idx[m] : m) * stride; idx points to shared memory (token ids -> embedding rows).
struct XSrc {
  const float* base;
  size_t stride;
  const int* idx;
  __device__ __forceinline__ const float* row(int m) const { return base + (size_t)(idx ? idx[m] : m) * stride; }
};

// Activation rows [M][klen] -> shared memory, fp32, row stride kcl + X_PAD floats.  The rows
// arrive by bulk async copies (one per row, all in flight together); columns klen..kcl are
// zeroed.  With NORM one pass over the tile accumulates sum(x^2), multiplies the RMSNorm
// gain in and leaves 1/rms in ctl->inv[m] for the epilogue (a per-row scalar commutes with
// the contraction).  `copy_out`: also publish the raw rows to global memory.
template <int M, bool NORM>
__device__ void load_x(float* X, int kcl, int klen, const XSrc& src, int k0, const float* norm_w, float eps,
                       int Ktotal, Ctrl* ctl, unsigned& xphase, float* copy_out, volatile int* err,
                       const float* ssq_in = nullptr, int G = 0) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int xs = kcl + X_PAD;
  if (tid == 0) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_arrive_expect_tx(&ctl->xbar, (unsigned)(M * klen * 4));
#pragma unroll
    for (int m = 0; m < M; ++m)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(X + m * xs)), "l"(src.row(m) + k0), "r"((unsigned)(klen * 4)),
                     "r"(smem_u32(&ctl->xbar))
                   : "memory");
  }
  // zero the padding columns meanwhile (weights are zero there, but 0 * garbage may be NaN)
  const int padq = (kcl - klen) >> 2;
  for (int i = tid; i < M * padq; i += CONSUMER_THREADS) {
    const int m = i / padq, c = i - m * padq;
    reinterpret_cast<float4*>(X + m * xs + klen)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  constexpr int PER = KC_MAX / 4 / CONSUMER_THREADS;
  const int kl4 = klen >> 2;
  float4 gain[PER];
  if (NORM) {   // the gains travel while the rows are still in flight
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int k4 = tid + i * CONSUMER_THREADS;
      gain[i] = k4 < kl4 ? __ldg(reinterpret_cast<const float4*>(norm_w) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  float part[8];
  if (!NORM && ssq_in && warp < M) {   // requested after the rows' copies were issued
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = lane + 32 * i;
      part[i] = c < G ? ldcg(ssq_in + c * 8 + warp) : 0.f;
    }
  }
  mbar_wait(&ctl->xbar, xphase, err, DEV_TIMEOUT_FULL);
  xphase ^= 1u;
  if (NORM) {
    float ss[M];
#pragma unroll
    for (int m = 0; m < M; ++m) ss[m] = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int k4 = tid + i * CONSUMER_THREADS;
      if (k4 < kl4) {
        const float4 g = gain[i];
#pragma unroll
        for (int m = 0; m < M; ++m) {
          float4* xp = reinterpret_cast<float4*>(X + m * xs) + k4;
          float4 x = *xp;
          if (copy_out) __stcg(reinterpret_cast<float4*>(copy_out + (size_t)m * Ktotal + (k4 << 2)), x);
          ss[m] += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
          x.x *= g.x; x.y *= g.y; x.z *= g.z; x.w *= g.w;
          *xp = x;
        }
      }
    }
#pragma unroll
    for (int m = 0; m < M; ++m) {
      float v = ss[m];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) ctl->red[warp][m] = v;
    }
    named_sync(1, CONSUMER_THREADS);
    if (tid < M) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += ctl->red[w][tid];
      ctl->inv[tid] = 1.0f / sqrtf(s / (float)Ktotal + eps);
    }
  } else if (ssq_in) {
    // the rows already carry the gain; the sums of squares wait as per-CTA partials (left by the last
    // residual epilogue): warp m adds them up for row m in a fixed order
    if (warp < M) {
      float v = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) v += part[i];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) ctl->inv[warp] = 1.0f / sqrtf(v / (float)Ktotal + eps);
    }
  } else if (tid < M) {
    ctl->inv[tid] = 1.0f;
  }
  named_sync(1, CONSUMER_THREADS);
}

// ------------------------------------------------------------------------------ reduction

// Sum each of CNT values over the 32 lanes.  While the count is a multiple of 4 the
// lanes split the values (half kept, half sent); afterwards every value is all-reduced.
// On return lane holds `final_cnt` sums starting at value index `base`.
template <int CNT, int BIT>
__device__ __forceinline__ void reduce_rec(float* v, int& base, int lane) {
  if constexpr (BIT > 0) {
    if constexpr (CNT % 4 == 0) {
      constexpr int HALF = CNT / 2;
      const bool up = (lane & BIT) != 0;
#pragma unroll
      for (int i = 0; i < HALF; ++i) {
        const float keep = up ? v[i + HALF] : v[i];
        const float send = up ? v[i] : v[i + HALF];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, BIT);
      }
      if (up) base += HALF;
      reduce_rec<HALF, BIT / 2>(v, base, lane);
    } else {
#pragma unroll
      for (int i = 0; i < CNT; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], BIT);
      reduce_rec<CNT, BIT / 2>(v, base, lane);
    }
  }
}
constexpr int final_cnt(int cnt, int bit) { return bit == 0 ? cnt : (cnt % 4 == 0 ? final_cnt(cnt / 2, bit / 2) : cnt); }
constexpr int dup_mask(int cnt, int bit) {
  return bit == 0 ? 0 : (cnt % 4 == 0 ? dup_mask(cnt / 2, bit / 2) : (bit | dup_mask(cnt, bit / 2)));
}

// ------------------------------------------------------------------------------ epilogues

struct EpiArgs {
  float* out;     // STORE: [M][ldo]; RESID: x [M][ldo]; SWIGLU: act [M][ldo]
  int ldo;
  // RESID on bf16 models: the epilogue also prepares the next RMSNorm (NULL: off)
  const float* next_gain;   // gain of the norm that reads the updated residual stream next
  float* xg;                // [M][ldo] = x * next_gain
  float* ssq;               // [grid][8] partial sums of x^2
  // QKV
  float* qbuf; void* kc; void* vc;  // cache bases already offset to the layer
  const float *cs, *sn;
  const int *rowslot, *rowpos;      // per activation row: cache row to append to, rotary position (shared memory)
  int d, dh, max_seq;
};

__device__ __forceinline__ void cache_store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void cache_store(float* p, float v) { *p = v; }

// (a, b) are the results of rows n and n+1 (n even) for activation row m.
template <typename WT>
__device__ __forceinline__ void epilogue_pair(int epi, const EpiArgs& e, int m, int n, int N, float a, float b) {
  if (n >= N) return;
  if (epi == EPI_STORE) {
    stcg(e.out + (size_t)m * e.ldo + n, a);
    if (n + 1 < N) stcg(e.out + (size_t)m * e.ldo + n + 1, b);
  } else if (epi == EPI_RESID) {
    float* p = e.out + (size_t)m * e.ldo + n;
    stcg(p, ldcg(p) + a);
    if (n + 1 < N) stcg(p + 1, ldcg(p + 1) + b);
  } else if (epi == EPI_SWIGLU) {
    const float s = a / (1.0f + expf(-a));
    stcg(e.out + (size_t)m * e.ldo + (n >> 1), s * b);
  } else {  // EPI_QKV: rows are [q | k | v]; q and k rows are stored pair-interleaved
    const int region = n / e.d, c = n - region * e.d;
    const int slot = e.rowslot[m];
    if (region == 2) {
      const int hv = c / e.dh;
      WT* vp = static_cast<WT*>(e.vc) + ((size_t)hv * e.max_seq + slot) * e.dh + (c - hv * e.dh);
      cache_store(vp, a);
      cache_store(vp + 1, b);
    } else {
      const int h = c / e.dh, i = (c - h * e.dh) >> 1, half = e.dh >> 1;
      const int pos = e.rowpos[m];
      const float cs = e.cs[pos * half + i], sn = e.sn[pos * half + i];
      const float ra = a * cs - b * sn, rb = b * cs + a * sn;
      const int c0 = h * e.dh + i;
      if (region == 0) {
        stcg(e.qbuf + (size_t)m * e.d + c0, ra);
        stcg(e.qbuf + (size_t)m * e.d + c0 + half, rb);
      } else {
        WT* kp = static_cast<WT*>(e.kc) + ((size_t)h * e.max_seq + slot) * e.dh + i;
        cache_store(kp, ra);
        cache_store(kp + half, rb);
      }
    }
  }
}

// ------------------------------------------------------------------------------ consumers

__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// fp32 weights: warp w owns rows 4w..4w+3 of the tile, lanes split K, packed fp32 FMAs.
template <int M>
__device__ __forceinline__ void compute_step_f32(const char* stage, const float* X, int xs, int s, int warp,
                                                 int lane, float2 (&acc)[4][M]) {
  const uint4* wp = reinterpret_cast<const uint4*>(stage + warp * 2048 + lane * 16);
  float2 w[4][2];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const uint4 q = wp[r * 32];
    w[r][0] = make_float2(__uint_as_float(q.x), __uint_as_float(q.y));
    w[r][1] = make_float2(__uint_as_float(q.z), __uint_as_float(q.w));
  }
#pragma unroll
  for (int m = 0; m < M; ++m) {
    const float4 xa = reinterpret_cast<const float4*>(X + m * xs)[s * 32 + lane];
    const float2 x0 = make_float2(xa.x, xa.y), x1 = make_float2(xa.z, xa.w);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float2 a = acc[r][m];
      a = __ffma2_rn(w[r][0], x0, a);
      a = __ffma2_rn(w[r][1], x1, a);
      acc[r][m] = a;
    }
  }
}

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// This CTA's share of one projection.  src gives the M activation rows (fp32).
template <int M, typename WT, bool TRACE>
__device__ void consume_gemm(const Gemm& g, const EpiArgs& e, const XSrc& src, const float* norm_w, float eps,
                             float* copy_out, const float* ssq_in, int cta, int G, Ring& ring, Ctrl* ctl, float* X,
                             unsigned& xphase, float* red, float* pre_s, uint32_t zero_addr, const char* stages, volatile int* err) {
  constexpr int EPL = WTraits<WT>::EPL, KSTEP = 32 * EPL;
  constexpr bool BF = sizeof(WT) == 2;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int q0, q1;
  cta_quads(g.N, cta, G, q0, q1);
  const int rows = (q1 - q0) * 4;
  if (rows == 0) {
    if (copy_out) {   // this CTA only has to publish the input rows (residual stream)
      for (int i = tid; i < M * (g.K >> 2); i += CONSUMER_THREADS) {
        const int m = i / (g.K >> 2), k = (i - m * (g.K >> 2)) << 2;
        __stcg(reinterpret_cast<float4*>(copy_out + (size_t)m * g.K + k),
               __ldcg(reinterpret_cast<const float4*>(src.row(m) + k)));
      }
    }
    if (e.ssq && tid < 8) stcg(e.ssq + cta * 8 + tid, 0.f);
    return;
  }
  int nchunk, kcl;
  chunking(g.K, KSTEP, nchunk, kcl);
  const int xs = kcl + X_PAD;
  if (nchunk == 1) {
    const bool prenorm = g.pro == PRO_NORM && ssq_in != nullptr;
    if (g.pro == PRO_NORM && !prenorm)
      load_x<M, true>(X, kcl, g.K, src, 0, norm_w, eps, g.K, ctl, xphase, copy_out, err);
    else
      load_x<M, false>(X, kcl, g.K, src, 0, nullptr, eps, g.K, ctl, xphase, nullptr, err, prenorm ? ssq_in : nullptr, G);
  }
  if constexpr (TRACE) trace_stamp(ctl, 1);
  const int gq = lane >> 2, tq = lane & 3;
  float ssq_acc = 0.f;    // threads 0..7: this CTA's sum of x^2 of activation row tid (bf16 RESID with xg)
  for (int t = 0; t * 32 < rows; ++t) {
    const int nr = min(32, rows - t * 32);
    const int n0 = q0 * 4 + t * 32;
    float2 acc[4][M];       // fp32 path
    float dacc[2][4];       // bf16 path: two 16-row groups x (16 rows x 8 columns) fragment
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int m = 0; m < M; ++m) acc[r][m] = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) dacc[i][j] = 0.f;
    // bf16 RESID: the residual values (and the next norm's gains) of this tile travel to shared
    // memory asynchronously while the K loop runs: pre_s[m*32 + row] and pre_s[256 + row].  No
    // register waits for them until the epilogue.
    if (BF && g.epi == EPI_RESID) {
      const int row = tid >> 3, m = tid & 7;
      if (m < M && (row & 3) == 0 && row < nr) cp_async16(pre_s + m * 32 + row, e.out + (size_t)m * e.ldo + n0 + row);
      if (e.xg && tid < 8 && tid * 4 < nr) cp_async16(pre_s + 256 + tid * 4, e.next_gain + n0 + tid * 4);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int c = 0; c < nchunk; ++c) {
      const int k0 = c * kcl, klen = min(kcl, g.K - k0);
      if (nchunk > 1) {
        named_sync(1, CONSUMER_THREADS);  // everyone is done with the previous chunk
        load_x<M, false>(X, kcl, klen, src, k0, nullptr, 0.f, g.K, ctl, xphase, nullptr, err);
      }
      for (int s = 0; s * KSTEP < klen; ++s) {
        mbar_wait(&ctl->full[ring.stage], ring.phase, err, DEV_TIMEOUT_FULL);
        const char* stage = stages + (size_t)ring.stage * STAGE_BYTES;
        if constexpr (!BF) {
          if (warp * 4 < nr) compute_step_f32<M>(stage, X, xs, s, warp, lane, acc);
        } else {
          // warp w takes the two 16-wide K slices 2w, 2w+1 of this 256-wide step
          const uint32_t st_addr = smem_u32(stage);
          const int mat = lane >> 3, rr = lane & 7;
          // B fragments from the fp32 tile, split on the fly: x = hi + lo (two bf16)
          uint32_t bq[2][4];
#pragma unroll
          for (int kk = 0; kk < 2; ++kk) {
            const int c16 = (warp * 2 + kk) * 2;     // first 16-byte chunk of the slice (of 32)
            float2 xa = make_float2(0.f, 0.f), xb = make_float2(0.f, 0.f);
            if (gq < M) {
              const float* xr = X + gq * xs + s * 256 + c16 * 8 + 2 * tq;
              xa = *reinterpret_cast<const float2*>(xr);
              xb = *reinterpret_cast<const float2*>(xr + 8);
            }
            bq[kk][0] = pack_bf16(xa.x, xa.y);
            bq[kk][1] = pack_bf16(xb.x, xb.y);
            bq[kk][2] = pack_bf16(xa.x - bf16lo(bq[kk][0]), xa.y - bf16hi(bq[kk][0]));
            bq[kk][3] = pack_bf16(xb.x - bf16lo(bq[kk][1]), xb.y - bf16hi(bq[kk][1]));
          }
          // A fragments of both slices and both 16-row groups first, then the eight MMAs
          uint32_t af[2][2][4];
#pragma unroll
          for (int kk = 0; kk < 2; ++kk) {
            const int c16 = (warp * 2 + kk) * 2;
#pragma unroll
            for (int gi = 0; gi < 2; ++gi) {
              // A: matrices {rows 0-7 k0-7, rows 8-15 k0-7, rows 0-7 k8-15, rows 8-15 k8-15}
              const int r = gi * 16 + (mat & 1) * 8 + rr;
              const int ch = (c16 + (mat >> 1)) ^ (r & 7);
              const uint32_t addr = r < nr ? st_addr + (uint32_t)(r * 512 + ch * 16) : zero_addr;
              if (gi * 16 < nr) ldsm4(addr, af[kk][gi][0], af[kk][gi][1], af[kk][gi][2], af[kk][gi][3]);
            }
          }
#pragma unroll
          for (int kk = 0; kk < 2; ++kk)
#pragma unroll
            for (int gi = 0; gi < 2; ++gi)
              if (gi * 16 < nr) {
                mma_bf16(dacc[gi], af[kk][gi][0], af[kk][gi][1], af[kk][gi][2], af[kk][gi][3], bq[kk][0], bq[kk][1]);
                mma_bf16(dacc[gi], af[kk][gi][0], af[kk][gi][1], af[kk][gi][2], af[kk][gi][3], bq[kk][2], bq[kk][3]);
              }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[ring.stage]);
        ring.advance();
      }
    }
    if constexpr (TRACE) { if (t * 32 + 32 >= rows) trace_stamp(ctl, 2); }
    if constexpr (!BF) {
      // 4*M sums per warp, value index m*4 + r
      float v[4 * M];
#pragma unroll
      for (int m = 0; m < M; ++m)
#pragma unroll
        for (int r = 0; r < 4; ++r) v[m * 4 + r] = acc[r][m].x + acc[r][m].y;
      int base = 0;
      reduce_rec<4 * M, 16>(v, base, lane);
      constexpr int FC = final_cnt(4 * M, 16), DUP = dup_mask(4 * M, 16);
      if ((lane & DUP) == 0 && warp * 4 < nr) {
#pragma unroll
        for (int i = 0; i < FC; i += 2) {
          const int vi = base + i, m = vi >> 2, r = vi & 3;
          const float sc = ctl->inv[m];
          epilogue_pair<WT>(g.epi, e, m, n0 + warp * 4 + r, g.N, v[i] * sc, v[i + 1] * sc);
        }
      }
    } else {
      // partial sums of the 8 warps (each had its own K slices) meet in shared memory
#pragma unroll
      for (int gi = 0; gi < 2; ++gi) {
        float* rp = red + ((warp * 2 + gi) * 16) * 8;
        *reinterpret_cast<float2*>(rp + gq * 8 + tq * 2) = make_float2(dacc[gi][0], dacc[gi][1]);
        *reinterpret_cast<float2*>(rp + (gq + 8) * 8 + tq * 2) = make_float2(dacc[gi][2], dacc[gi][3]);
      }
      if (g.epi == EPI_RESID) asm volatile("cp.async.wait_group 0;" ::: "memory");
      named_sync(1, CONSUMER_THREADS);
      {
        // thread -> (row of the tile, activation row): tid = row*8 + m
        float resid = 0.f, gnext = 0.f;
        if (g.epi == EPI_RESID) {
          resid = pre_s[(tid & 7) * 32 + (tid >> 3)];
          gnext = pre_s[256 + (tid >> 3)];
        }
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[w * 256 + tid];
        const int row = tid >> 3, m = tid & 7;
        v = v * ctl->inv[m < M ? m : 0] + resid;
        const float partner = __shfl_down_sync(0xffffffffu, v, 8);
        if ((row & 1) == 0 && m < M && row < nr)
          epilogue_pair<WT>(g.epi == EPI_RESID ? EPI_STORE : g.epi, e, m, n0 + row, g.N, v, partner);
        if (g.epi == EPI_RESID && e.xg) {
          // v is the updated residual stream at (m, n0 + row): hand the next RMSNorm its input
          // times the gain, and this warp's share of sum(x^2) per activation row
          const bool valid = m < M && row < nr && n0 + row < g.N;
          if (valid) stcg(e.xg + (size_t)m * e.ldo + n0 + row, v * gnext);
          float sq = valid ? v * v : 0.f;
          sq += __shfl_xor_sync(0xffffffffu, sq, 8);
          sq += __shfl_xor_sync(0xffffffffu, sq, 16);
          if (lane < 8) ctl->red[warp][lane] = sq;
        }
      }
      named_sync(1, CONSUMER_THREADS);
      if (g.epi == EPI_RESID && e.xg && tid < 8) {
#pragma unroll
        for (int w = 0; w < 8; ++w) ssq_acc += ctl->red[w][tid];
      }
    }
  }
  if (BF && g.epi == EPI_RESID && e.ssq && tid < 8) stcg(e.ssq + cta * 8 + tid, ssq_acc);
}

// ------------------------------------------------------------------------------ grid barrier

__device__ __forceinline__ void grid_barrier(unsigned* counter, unsigned& target, unsigned G, volatile int* err,
                                             unsigned limit = SPIN_LIMIT_GRID) {
  named_sync(1, CONSUMER_THREADS);
  if (threadIdx.x == 0) {
    target += G;
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
    unsigned it = 0;
    while (ld_acquire(counter) < target) {
      if (++it > limit || ((it & 255u) == 0 && *err != DEV_OK)) {
        atomicCAS(const_cast<int*>(err), DEV_OK, DEV_TIMEOUT_GRID);
        break;
      }
    }
    // no fence here: the acquire load above orders this thread, the CTA barrier below hands
    // that order on to the other compute threads (cumulativity)
  }
  named_sync(1, CONSUMER_THREADS);
}

// The same barrier for a grid that is one thread-block cluster: the first G threads each arrive
// on the barrier word in one member's shared memory, thread 0 waits for the G arrivals on its
// own.  Release / acquire at cluster scope order the global-memory traffic around it like the
// red.release / ld.acquire pair above does at gpu scope; the cost is a hop between SMs instead
// of two trips to L2.
__device__ __forceinline__ void cluster_barrier(uint64_t* cbar, unsigned& phase, unsigned G, volatile int* err,
                                                unsigned limit = SPIN_LIMIT_GRID) {
  named_sync(1, CONSUMER_THREADS);
  if (threadIdx.x < G) mbar_arrive_remote(cluster_map(smem_u32(cbar), threadIdx.x));
  if (threadIdx.x == 0) {
    unsigned it = 0;
    while (!mbar_try_wait_cluster(cbar, phase)) {
      if (++it > limit || ((it & 255u) == 0 && *err != DEV_OK)) {
        atomicCAS(const_cast<int*>(err), DEV_OK, DEV_TIMEOUT_GRID);
        break;
      }
    }
  }
  phase ^= 1u;
  named_sync(1, CONSUMER_THREADS);
}

// ------------------------------------------------------------------------------ attention

template <typename CT> struct CTraits;
template <> struct CTraits<__nv_bfloat16> {
  static constexpr int E = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
    const uint4 r = __ldcg(reinterpret_cast<const uint4*>(p));
    f[0] = bf16lo(r.x); f[1] = bf16hi(r.x); f[2] = bf16lo(r.y); f[3] = bf16hi(r.y);
    f[4] = bf16lo(r.z); f[5] = bf16hi(r.z); f[6] = bf16lo(r.w); f[7] = bf16hi(r.w);
  }
};
template <> struct CTraits<float> {
  static constexpr int E = 4;
  static __device__ __forceinline__ void load(const float* p, float (&f)[4]) {
    const float4 r = __ldcg(reinterpret_cast<const float4*>(p));
    f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w;
  }
};

// Merge of a head's KV splits (run by the CTA that finished the head's last split): the
// per-split maxima and sums are fetched once into shared memory and turned into weights
// w_s = exp(max_s - max) / sum_s' w_s' sum_s'; the partial outputs are then combined with all
// loads of a thread in flight together.
template <int M>
__device__ void merge_head(const ModelDev& md, int h, int nsplit, float* scratch) {
  const int tid = threadIdx.x, dh = md.dh, d = md.d;
  float* mxs = scratch;                   // [nsplit][M] max, then weight
  float* sms = scratch + nsplit * M;      // [nsplit][M] sum
  for (int i = tid; i < nsplit * M; i += CONSUMER_THREADS) {
    const int s2 = i / M, m = i - s2 * M;
    const float* ml = md.aml + ((size_t)(h * nsplit + s2) * MAX_M + m) * 2;
    mxs[i] = ldcg(ml);
    sms[i] = ldcg(ml + 1);
  }
  named_sync(1, CONSUMER_THREADS);
  if (tid < M) {
    float gmax = -INFINITY;
    for (int s2 = 0; s2 < nsplit; ++s2) gmax = fmaxf(gmax, mxs[s2 * M + tid]);
    float den = 0.f;
    for (int s2 = 0; s2 < nsplit; ++s2) {
      const float mx = mxs[s2 * M + tid];
      const float w = (mx == -INFINITY) ? 0.f : expf(mx - gmax);
      den = fmaf(w, sms[s2 * M + tid], den);
      mxs[s2 * M + tid] = w;
    }
    const float inv = 1.0f / den;
    for (int s2 = 0; s2 < nsplit; ++s2) mxs[s2 * M + tid] *= inv;
  }
  named_sync(1, CONSUMER_THREADS);
  for (int i = tid; i < M * dh; i += CONSUMER_THREADS) {
    const int m = i / dh, c = i - m * dh;
    float num = 0.f;
    for (int s0 = 0; s0 < nsplit; s0 += 4) {
      float pv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        pv[u] = (s0 + u < nsplit) ? ldcg(md.apart + ((size_t)(h * nsplit + s0 + u) * MAX_M) * dh + i) : 0.f;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (s0 + u < nsplit) num = fmaf(mxs[(s0 + u) * M + m], pv[u], num);
    }
    stcg(md.attn + (size_t)m * d + h * dh + c, num);
  }
  if (tid == 0) md.head_cnt[h] = 0u;
}


template <typename CT>
__device__ __forceinline__ void frag_from_smem(const char* p, float (&f)[CTraits<CT>::E]) {
  const uint4 r = *reinterpret_cast<const uint4*>(p);
  if constexpr (sizeof(CT) == 2) {
    f[0] = bf16lo(r.x); f[1] = bf16hi(r.x); f[2] = bf16lo(r.y); f[3] = bf16hi(r.y);
    f[4] = bf16lo(r.z); f[5] = bf16hi(r.z); f[6] = bf16lo(r.w); f[7] = bf16hi(r.w);
  } else {
    f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y); f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
  }
}

// Query row m attends every cache row below `origin` and, of the `nslots` rows from the origin
// on, those named in ctl->sees[m] (a chain: rows origin..origin+m).  Work unit = (head, KV
// split).  The unit's K and V rows are brought into shared memory with asynchronous
// 16-byte copies, all in flight at once (one memory latency), in sub-chunks that fit the
// scratch region, with a running (online) softmax across sub-chunks.  Each unit leaves an
// unnormalised partial output with its row max and sum; the CTA that finishes a head's
// last split merges them (no waiting).
template <int M, typename CT>
__device__ void attn_phase(const ModelDev& md, int layer, int origin, int nslots, int cta, int G, char* xs, int xbytes,
                           Ctrl* ctl) {
  constexpr int E = CTraits<CT>::E;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = md.H, dh = md.dh, d = md.d;
  const int len = origin + nslots;
  const int nsplit = eff_nsplit(md, len);
  const int Lc = (len + nsplit - 1) / nsplit;
  const int LPP = dh / E, PPI = 32 / LPP;
  const int sub = lane / LPP, li = lane - sub * LPP;
  const int rowb = dh * (int)sizeof(CT);                     // bytes of one head row
  // scratch: q [M][dh] | K tile [SC][rowb] (later the cross-warp buffer) | V tile | S [M][SC]
  int SC = (xbytes - M * dh * 4) / (2 * rowb + M * 4);
  SC = min(SC & ~7, (Lc + 7) & ~7);
  float* qs = reinterpret_cast<float*>(xs);
  char* Kt = xs + M * dh * 4;
  char* Vt = Kt + (size_t)SC * rowb;
  float* S = reinterpret_cast<float*>(Vt + (size_t)SC * rowb);
  float* red = reinterpret_cast<float*>(Kt);                 // [8][M][dh], needs SC*rowb >= 32*M*dh
  const CT* Kl = static_cast<const CT*>(md.kcache) + (size_t)layer * md.max_seq * d;
  const CT* Vl = static_cast<const CT*>(md.vcache) + (size_t)layer * md.max_seq * d;
  const int cpr = rowb >> 4;                                  // 16-byte copies per row

  for (int unit = cta; unit < H * nsplit; unit += G) {
    const int h = unit / nsplit, sp = unit - h * nsplit;
    const int p0 = sp * Lc, p1 = min(len, p0 + Lc);
    for (int i = tid; i < M * dh; i += CONSUMER_THREADS) {
      const int m = i / dh, c = i - m * dh;
      qs[i] = ldcg(md.qbuf + (size_t)m * d + h * dh + c) * md.scale;
    }
    if (tid < M) { ctl->rowmax[tid] = -INFINITY; ctl->rowsum[tid] = 0.f; }
    float acc[M][E];
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
      for (int e = 0; e < E; ++e) acc[m][e] = 0.f;
    named_sync(1, CONSUMER_THREADS);
    float qr[M][E];
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
      for (int e = 0; e < E; ++e) qr[m][e] = qs[m * dh + li * E + e];

    for (int c0 = p0; c0 < p1; c0 += SC) {
      const int n = min(SC, p1 - c0);
      for (int i = tid; i < n * cpr; i += CONSUMER_THREADS) {
        const int r = i / cpr, cc = i - r * cpr;
        const size_t g = (((size_t)h * md.max_seq + c0 + r) * dh) * sizeof(CT) + (size_t)cc * 16;
        cp_async16(Kt + (size_t)r * rowb + cc * 16, reinterpret_cast<const char*>(Kl) + g);
        cp_async16(Vt + (size_t)r * rowb + cc * 16, reinterpret_cast<const char*>(Vl) + g);
      }
      cp_async_wait_all();
      named_sync(1, CONSUMER_THREADS);
      // scores
      for (int pb = warp * PPI; pb < n; pb += 8 * PPI) {
        const int r = pb + sub;
        float kf[E];
#pragma unroll
        for (int e = 0; e < E; ++e) kf[e] = 0.f;
        if (r < n) frag_from_smem<CT>(Kt + (size_t)r * rowb + li * 16, kf);
        float part[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
          float sacc = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) sacc = fmaf(kf[e], qr[m][e], sacc);
          part[m] = sacc;
        }
        for (int o = LPP >> 1; o; o >>= 1)
#pragma unroll
          for (int m = 0; m < M; ++m) part[m] += __shfl_xor_sync(0xffffffffu, part[m], o);
        if (r < n && li == 0) {
#pragma unroll
          for (int m = 0; m < M; ++m) {
            const int rel = c0 + r - origin;
            S[m * SC + r] = (rel < 0 || ((ctl->sees[m] >> rel) & 1u)) ? part[m] : -INFINITY;
          }
        }
      }
      named_sync(1, CONSUMER_THREADS);
      // online softmax: warp m owns row m
      if (warp < M) {
        float* row = S + warp * SC;
        float mx = -INFINITY;
        for (int i = lane; i < n; i += 32) mx = fmaxf(mx, row[i]);
#pragma unroll
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float old = ctl->rowmax[warp];
        const float nm = fmaxf(old, mx);
        float sum = 0.f;
        for (int i = lane; i < n; i += 32) {
          const float ex = (nm == -INFINITY) ? 0.f : expf(row[i] - nm);
          row[i] = ex;
          sum += ex;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) {
          const float rescale = (old == -INFINITY) ? 0.f : expf(old - nm);
          ctl->red[0][warp] = rescale;
          ctl->rowsum[warp] = ctl->rowsum[warp] * rescale + sum;
          ctl->rowmax[warp] = nm;
        }
      }
      named_sync(1, CONSUMER_THREADS);
      // rescale what was accumulated so far, add this sub-chunk's weighted V rows
#pragma unroll
      for (int m = 0; m < M; ++m) {
        const float rs = ctl->red[0][m];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[m][e] *= rs;
      }
      for (int pb = warp * PPI; pb < n; pb += 8 * PPI) {
        const int r = pb + sub;
        if (r < n) {
          float vf[E];
          frag_from_smem<CT>(Vt + (size_t)r * rowb + li * 16, vf);
#pragma unroll
          for (int m = 0; m < M; ++m) {
            const float w = S[m * SC + r];
#pragma unroll
            for (int e = 0; e < E; ++e) acc[m][e] = fmaf(w, vf[e], acc[m][e]);
          }
        }
      }
      named_sync(1, CONSUMER_THREADS);   // tiles and S are free again
    }
    for (int o = LPP; o < 32; o <<= 1)
#pragma unroll
      for (int m = 0; m < M; ++m)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[m][e] += __shfl_xor_sync(0xffffffffu, acc[m][e], o);
    if (sub == 0) {
#pragma unroll
      for (int m = 0; m < M; ++m)
#pragma unroll
        for (int e = 0; e < E; ++e) red[(warp * M + m) * dh + li * E + e] = acc[m][e];
    }
    named_sync(1, CONSUMER_THREADS);
    if (nsplit == 1) {   // the whole context was here: normalise and finish the head
      for (int i = tid; i < M * dh; i += CONSUMER_THREADS) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[w * M * dh + i];
        const int m = i / dh, c = i - m * dh;
        stcg(md.attn + (size_t)m * d + h * dh + c, s / ctl->rowsum[m]);
      }
      named_sync(1, CONSUMER_THREADS);
      continue;
    }
    float* part_out = md.apart + ((size_t)(h * nsplit + sp) * MAX_M) * dh;
    for (int i = tid; i < M * dh; i += CONSUMER_THREADS) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += red[w * M * dh + i];
      stcg(part_out + i, s);
    }
    if (tid < M) {
      float* ml = md.aml + ((size_t)(h * nsplit + sp) * MAX_M + tid) * 2;
      stcg(ml, ctl->rowmax[tid]);
      stcg(ml + 1, ctl->rowsum[tid]);
    }
    __threadfence();
    named_sync(1, CONSUMER_THREADS);
    if (tid == 0) {
      const unsigned old = atomicAdd(md.head_cnt + h, 1u);
      ctl->flag = (old == (unsigned)nsplit - 1u);
      __threadfence();
    }
    named_sync(1, CONSUMER_THREADS);
    if (ctl->flag) merge_head<M>(md, h, nsplit, reinterpret_cast<float*>(Kt));
    named_sync(1, CONSUMER_THREADS);
  }
}

__device__ __forceinline__ void ldsm4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// split two fp32 pairs into bf16 hi and lo B-fragment registers
__device__ __forceinline__ void split_frag(float2 xa, float2 xb, uint32_t& h0, uint32_t& h1, uint32_t& l0, uint32_t& l1) {
  h0 = pack_bf16(xa.x, xa.y);
  h1 = pack_bf16(xb.x, xb.y);
  l0 = pack_bf16(xa.x - bf16lo(h0), xa.y - bf16hi(h0));
  l1 = pack_bf16(xb.x - bf16lo(h1), xb.y - bf16hi(h1));
}

// Piece i of a K/V tile -> (row, 16-byte piece of the row).  The long units of the batched kernel
// (SHIFT) use the fact that a row has a power-of-two number of pieces; the decode kernel keeps
// the division (its instruction stream is left exactly as it was measured).
template <bool SHIFT>
__device__ __forceinline__ void piece_of(int i, int cpr, int csh, int& r, int& cc) {
  if constexpr (SHIFT) { r = i >> csh; cc = i & (cpr - 1); }
  else { r = i / cpr; cc = i - r * cpr; }
}

// bf16 KV cache: the same unit / split / merge scheme as attn_phase, with both products on
// the tensor cores.  Scores: D[16 positions x 8 queries] = K tile (A, ldmatrix) x q^T (B,
// fp32 q split into bf16 hi + lo).  Output: D[16 dims x 8 queries] = V^T (A, transposing
// ldmatrix) x P^T (B, fp32 probabilities split the same way); warp w owns dims 16w..16w+15,
// so no cross-warp reduction is needed.  Tile rows are 16-byte-chunk swizzled by position.
// PIPE (the batched kernel, where a unit spans several sub-chunks): two K/V tile buffers, the
// next sub-chunk's rows are requested before the current one is computed; with o_hi / o_lo the
// head's output rows [M][d] also leave as bf16 hi + lo (the next GEMM's operand).
template <int M, bool PIPE = false>
__device__ void attn_phase_mma(const ModelDev& md, int layer, int origin, int nslots, int cta, int G, char* xs,
                               int xbytes, Ctrl* ctl, __nv_bfloat16* o_hi = nullptr, __nv_bfloat16* o_lo = nullptr) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = md.H, dh = md.dh, d = md.d;
  const int len = origin + nslots;
  const int nsplit = eff_nsplit(md, len);
  const int Lc = (len + nsplit - 1) / nsplit;
  const int rowb = dh * 2, cpr = rowb >> 4;
  const int gq = lane >> 2, tq = lane & 3, mat = lane >> 3, rr = lane & 7;
  const int qst = dh + 8;                                    // padded fp32 row of q
  const char* Kl = static_cast<const char*>(md.kcache) + (size_t)layer * md.max_seq * d * 2;
  const char* Vl = static_cast<const char*>(md.vcache) + (size_t)layer * md.max_seq * d * 2;
  // scratch: q [M][dh+8] fp32 | NB x (K tile [SC][rowb] | V tile [SC][rowb]) | S [M][SC+8] fp32
  // PIPE also keeps q and the probabilities as packed bf16 (hi, lo) pairs -- the B fragments of the
  // MMAs as they are -- so that the fp32 -> hi/lo split is done once per unit / per probability
  // instead of once per use: + Qh | Ql [M][dh/2+4] words behind q, + Ph | Pl [M][SC/2+4] words behind S
  constexpr int NB = PIPE ? 2 : 1;
  const int qw = (dh >> 1) + 4;                              // words per packed q row
  const int qpk = PIPE ? 2 * M * qw * 4 : 0;
  int SC = ((xbytes - M * qst * 4 - qpk - M * 8 * 4 - (PIPE ? M * 8 * 4 : 0)) / (2 * NB * rowb + M * (PIPE ? 8 : 4))) & ~15;
  {  // equal sub-chunks instead of full ones plus a sliver
    const int nsub = (Lc + SC - 1) / SC;
    SC = min(SC, (((Lc + nsub - 1) / nsub) + 15) & ~15);
  }
  const int sst = SC + 8, pw = (SC >> 1) + 4;                // fp32 row of S, words per packed probability row
  float* qs = reinterpret_cast<float*>(xs);
  uint32_t* Qh = reinterpret_cast<uint32_t*>(xs + M * qst * 4);
  uint32_t* Ql = Qh + M * qw;
  char* const Kt0 = xs + M * qst * 4 + qpk;
  const size_t tileb = (size_t)SC * rowb;
  float* S = reinterpret_cast<float*>(Kt0 + 2 * NB * tileb);
  uint32_t* Ph = reinterpret_cast<uint32_t*>(S + M * sst);
  uint32_t* Pl = Ph + M * pw;
  // request rows [c0, c0 + n) of the head's K and V into tile buffer `buf`
  auto request = [&](int h, int c0, int n, int buf) {
    char* Kt = Kt0 + (size_t)buf * 2 * tileb;
    char* Vt = Kt + tileb;
    const int n16 = (n + 15) & ~15;
    const int csh = 31 - __clz(cpr);     // 16-byte pieces per row: a power of two
    for (int i = tid; i < n16 * cpr; i += CONSUMER_THREADS) {
      int r, cc;
      piece_of<PIPE>(i, cpr, csh, r, cc);
      const int dst = r * rowb + ((cc ^ (r & 7)) << 4);
      if (r < n) {
        const size_t g = (((size_t)h * md.max_seq + c0 + r) * dh) * 2 + (size_t)cc * 16;
        cp_async16(Kt + dst, Kl + g);
        cp_async16(Vt + dst, Vl + g);
      } else {   // rows past the end must not hold NaN patterns: P is 0 there
        *reinterpret_cast<uint4*>(Vt + dst) = make_uint4(0, 0, 0, 0);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const int nkd = dh >> 4;                                   // 16-wide slices of the head dim

  for (int unit = cta; unit < H * nsplit; unit += G) {
    const int h = unit / nsplit, sp = unit - h * nsplit;
    const int p0 = sp * Lc, p1 = min(len, p0 + Lc);
    // q rows (fp32) and the first sub-chunk of K/V are requested together
    for (int i = tid; i < M * (dh >> 2); i += CONSUMER_THREADS) {
      const int m = i / (dh >> 2), c = i - m * (dh >> 2);
      cp_async16(qs + m * qst + c * 4, md.qbuf + (size_t)m * d + h * dh + c * 4);
    }
    if (tid < M) { ctl->rowmax[tid] = -INFINITY; ctl->rowsum[tid] = 0.f; }
    float oacc[4] = {0.f, 0.f, 0.f, 0.f};
    int buf = 0;
    if (PIPE) request(h, p0, min(SC, p1 - p0), 0);
    for (int c0 = p0; c0 < p1; c0 += SC) {
      const int n = min(SC, p1 - c0), n16 = (n + 15) & ~15;
      if (PIPE) {
        const int c1 = c0 + SC;
        if (c1 < p1) {
          request(h, c1, min(SC, p1 - c1), buf ^ 1);
          asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
          asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
      } else {
        request(h, c0, n, 0);
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
      char* Kt = Kt0 + (size_t)buf * 2 * tileb;
      char* Vt = Kt + tileb;
      named_sync(1, CONSUMER_THREADS);
      if constexpr (PIPE) {
        if (c0 == p0) {   // q has arrived with the first sub-chunk: split it once for the whole unit
          for (int i = tid; i < M * (dh >> 1); i += CONSUMER_THREADS) {
            const int m = i / (dh >> 1), j = i - m * (dh >> 1);
            const float2 x = *reinterpret_cast<const float2*>(qs + m * qst + 2 * j);
            const uint32_t hq = pack_bf16(x.x, x.y);
            Qh[m * qw + j] = hq;
            Ql[m * qw + j] = pack_bf16(x.x - bf16lo(hq), x.y - bf16hi(hq));
          }
          named_sync(1, CONSUMER_THREADS);
        }
      }
      // ---- scores: warp takes 16-position groups
      for (int gp = warp; gp * 16 < n; gp += 8) {
        float dsc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int kd = 0; kd < nkd; ++kd) {
          uint32_t b0 = 0, b1 = 0, b2 = 0, b3 = 0;
          if constexpr (PIPE) {
            if (gq < M) {
              const int w = gq * qw + kd * 8 + tq;
              b0 = Qh[w]; b1 = Qh[w + 4]; b2 = Ql[w]; b3 = Ql[w + 4];
            }
          } else {
            float2 xa = make_float2(0.f, 0.f), xb = make_float2(0.f, 0.f);
            if (gq < M) {
              const float* qr = qs + gq * qst + kd * 16 + 2 * tq;
              xa = *reinterpret_cast<const float2*>(qr);
              xb = *reinterpret_cast<const float2*>(qr + 8);
            }
            split_frag(xa, xb, b0, b1, b2, b3);
          }
          const int r = gp * 16 + (mat & 1) * 8 + rr;
          const int ch = (kd * 2 + (mat >> 1)) ^ (r & 7);
          uint32_t a0, a1, a2, a3;
          ldsm4(smem_u32(Kt + r * rowb + ch * 16), a0, a1, a2, a3);
          mma_bf16(dsc, a0, a1, a2, a3, b0, b1);
          mma_bf16(dsc, a0, a1, a2, a3, b2, b3);
        }
        // dsc[0,1]: position gp*16+gq, queries 2tq, 2tq+1; dsc[2,3]: position +8
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = gp * 16 + gq + (j >> 1) * 8, q = 2 * tq + (j & 1);
          if (q < M) {
            const int rel = c0 + r - origin;
            const bool vis = r < n && (rel < 0 || ((ctl->sees[q] >> rel) & 1u));
            S[q * sst + r] = vis ? dsc[j] * md.scale : -INFINITY;
          }
        }
      }
      named_sync(1, CONSUMER_THREADS);
      // ---- online softmax: warp m owns row m
      if (warp < M) {
        float* row = S + warp * sst;
        float mx = -INFINITY;
        for (int i = lane; i < n16; i += 32) mx = fmaxf(mx, row[i]);
#pragma unroll
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float old = ctl->rowmax[warp];
        const float nm = fmaxf(old, mx);
        float sum = 0.f;
        if constexpr (PIPE) {   // probabilities leave as packed (hi, lo) pairs of two positions
          for (int i = 2 * lane; i < n16; i += 64) {
            const float2 sv = *reinterpret_cast<const float2*>(row + i);
            const float e0 = (nm == -INFINITY) ? 0.f : expf(sv.x - nm), e1 = (nm == -INFINITY) ? 0.f : expf(sv.y - nm);
            const uint32_t hp = pack_bf16(e0, e1);
            Ph[warp * pw + (i >> 1)] = hp;
            Pl[warp * pw + (i >> 1)] = pack_bf16(e0 - bf16lo(hp), e1 - bf16hi(hp));
            sum += e0 + e1;
          }
        } else {
          for (int i = lane; i < n16; i += 32) {
            const float ex = (nm == -INFINITY) ? 0.f : expf(row[i] - nm);
            row[i] = ex;
            sum += ex;
          }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) {
          const float rescale = (old == -INFINITY) ? 0.f : expf(old - nm);
          ctl->red[0][warp] = rescale;
          ctl->rowsum[warp] = ctl->rowsum[warp] * rescale + sum;
          ctl->rowmax[warp] = nm;
        }
      }
      named_sync(1, CONSUMER_THREADS);
      // ---- output: warp w owns dims 16w..16w+15 (warps beyond dh/16 idle)
      if (warp < nkd) {
        const float r0s = 2 * tq < M ? ctl->red[0][2 * tq] : 0.f, r1s = 2 * tq + 1 < M ? ctl->red[0][2 * tq + 1] : 0.f;
        oacc[0] *= r0s; oacc[1] *= r1s; oacc[2] *= r0s; oacc[3] *= r1s;
        for (int kp = 0; kp * 16 < n; ++kp) {
          uint32_t b0 = 0, b1 = 0, b2 = 0, b3 = 0;
          if constexpr (PIPE) {
            if (gq < M) {
              const int w = gq * pw + kp * 8 + tq;
              b0 = Ph[w]; b1 = Ph[w + 4]; b2 = Pl[w]; b3 = Pl[w + 4];
            }
          } else {
            float2 xa = make_float2(0.f, 0.f), xb = make_float2(0.f, 0.f);
            if (gq < M) {
              const float* pr = S + gq * sst + kp * 16 + 2 * tq;
              xa = *reinterpret_cast<const float2*>(pr);
              xb = *reinterpret_cast<const float2*>(pr + 8);
            }
            split_frag(xa, xb, b0, b1, b2, b3);
          }
          // A = V^T: matrices {pos 0-7 x dims 0-7, pos 0-7 x dims 8-15, pos 8-15 x dims 0-7, pos 8-15 x dims 8-15}
          const int r = kp * 16 + (mat >> 1) * 8 + rr;
          const int ch = (warp * 2 + (mat & 1)) ^ (r & 7);
          uint32_t a0, a1, a2, a3;
          ldsm4_trans(smem_u32(Vt + r * rowb + ch * 16), a0, a1, a2, a3);
          mma_bf16(oacc, a0, a1, a2, a3, b0, b1);
          mma_bf16(oacc, a0, a1, a2, a3, b2, b3);
        }
      }
      named_sync(1, CONSUMER_THREADS);   // tiles and S are free again
      if (PIPE) buf ^= 1;
    }
    // oacc[0,1]: dim 16w+gq, queries 2tq, 2tq+1; oacc[2,3]: dim +8
    if (nsplit == 1) {   // the whole context was here: normalise and finish the head
      if (warp < nkd) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int q = 2 * tq + (j & 1), c = warp * 16 + gq + (j >> 1) * 8;
          if (q < M) {
            const float v = oacc[j] / ctl->rowsum[q];
            if constexpr (PIPE) {
              if (o_hi) {
                const __nv_bfloat16 hv = __float2bfloat16_rn(v);
                o_hi[(size_t)q * d + h * dh + c] = hv;
                o_lo[(size_t)q * d + h * dh + c] = __float2bfloat16_rn(v - __bfloat162float(hv));
              } else {
                stcg(md.attn + (size_t)q * d + h * dh + c, v);
              }
            } else {
              stcg(md.attn + (size_t)q * d + h * dh + c, v);
            }
          }
        }
      }
      named_sync(1, CONSUMER_THREADS);
      continue;
    }
    float* part_out = md.apart + ((size_t)(h * nsplit + sp) * MAX_M) * dh;
    if (warp < nkd) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int q = 2 * tq + (j & 1), c = warp * 16 + gq + (j >> 1) * 8;
        if (q < M) stcg(part_out + q * dh + c, oacc[j]);
      }
    }
    if (tid < M) {
      float* ml = md.aml + ((size_t)(h * nsplit + sp) * MAX_M + tid) * 2;
      stcg(ml, ctl->rowmax[tid]);
      stcg(ml + 1, ctl->rowsum[tid]);
    }
    __threadfence();
    named_sync(1, CONSUMER_THREADS);
    if (tid == 0) {
      const unsigned old = atomicAdd(md.head_cnt + h, 1u);
      ctl->flag = (old == (unsigned)nsplit - 1u);
      __threadfence();
    }
    named_sync(1, CONSUMER_THREADS);
    if (ctl->flag) merge_head<M>(md, h, nsplit, reinterpret_cast<float*>(Kt0));
    named_sync(1, CONSUMER_THREADS);
    if constexpr (PIPE) {
      if (ctl->flag && o_hi) {   // the merged rows of this head, once more as bf16 hi + lo
        for (int i = tid; i < M * dh; i += CONSUMER_THREADS) {
          const int m = i / dh, c = i - m * dh;
          const float v = ldcg(md.attn + (size_t)m * d + h * dh + c);
          const __nv_bfloat16 hv = __float2bfloat16_rn(v);
          o_hi[(size_t)m * d + h * dh + c] = hv;
          o_lo[(size_t)m * d + h * dh + c] = __float2bfloat16_rn(v - __bfloat162float(hv));
        }
        named_sync(1, CONSUMER_THREADS);
      }
    }
  }
}

// ------------------------------------------------------------------------------ sampling

// Row statistics of logits/T over a slice of the vocabulary, one slice per CTA.
template <int M>
__device__ void stats_phase(const float* logits, int V, int rows0, int nrows, float temperature, int cta, int G,
                            float* stat_part, Ctrl* ctl) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int VS = (V + G - 1) / G;
  const int k0 = cta * VS, k1 = min(V, k0 + VS);
  for (int r = 0; r < nrows; ++r) {
    const float* row = logits + (size_t)(rows0 + r) * V;
    float mx = -INFINITY, av = -INFINITY;
    int ai = 0x7fffffff;
    for (int k = k0 + tid; k < k1; k += CONSUMER_THREADS) {
      const float l = ldcg(row + k);
      const float s = __fdiv_rn(l, temperature);
      mx = fmaxf(mx, s);
      if (l > av || ai == 0x7fffffff) { av = l; ai = k; }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float ov = __shfl_xor_sync(0xffffffffu, av, o);
      const int oi = __shfl_xor_sync(0xffffffffu, ai, o);
      if (oi != 0x7fffffff && (ai == 0x7fffffff || ov > av || (ov == av && oi < ai))) { av = ov; ai = oi; }
    }
    if (lane == 0) { ctl->sc.fval[warp] = mx; ctl->sc.amax[warp] = av; ctl->sc.aidx[warp] = ai; }
    named_sync(1, CONSUMER_THREADS);
    float cmx = -INFINITY;
#pragma unroll
    for (int w = 0; w < 8; ++w) cmx = fmaxf(cmx, ctl->sc.fval[w]);
    float sum = 0.f;
    for (int k = k0 + tid; k < k1; k += CONSUMER_THREADS)
      sum += expf(__fdiv_rn(ldcg(row + k), temperature) - cmx);
#pragma unroll
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    named_sync(1, CONSUMER_THREADS);
    if (lane == 0) ctl->sc.fval[warp] = sum;
    named_sync(1, CONSUMER_THREADS);
    if (tid == 0) {
      float tot = 0.f;
      float bv = ctl->sc.amax[0];
      int bi = ctl->sc.aidx[0];
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        tot += ctl->sc.fval[w];
        const int oi = ctl->sc.aidx[w];
        if (oi != 0x7fffffff && (bi == 0x7fffffff || ctl->sc.amax[w] > bv || (ctl->sc.amax[w] == bv && oi < bi))) {
          bv = ctl->sc.amax[w];
          bi = oi;
        }
      }
      float* o = stat_part + ((size_t)cta * MAX_M + r) * 4;
      stcg(o, cmx); stcg(o + 1, tot); stcg(o + 2, bv); stcg(o + 3, __int_as_float(bi));
    }
    named_sync(1, CONSUMER_THREADS);
  }
}

// Merge the per-CTA slices: row max, sum of exp, argmax (lowest index on ties).
__device__ void merge_stats(const float* stat_part, int G, int nrows, Ctrl* ctl, float* rmax, float* rsum,
                            int* rarg) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (warp < nrows) {
    const int r = warp;
    float mx = -INFINITY, av = -INFINITY;
    int ai = 0x7fffffff;
    for (int c = lane; c < G; c += 32) {
      const float* o = stat_part + ((size_t)c * MAX_M + r) * 4;
      mx = fmaxf(mx, ldcg(o));
      const float ov = ldcg(o + 2);
      const int oi = __float_as_int(ldcg(o + 3));
      if (oi != 0x7fffffff && (ai == 0x7fffffff || ov > av || (ov == av && oi < ai))) { av = ov; ai = oi; }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float ov = __shfl_xor_sync(0xffffffffu, av, o);
      const int oi = __shfl_xor_sync(0xffffffffu, ai, o);
      if (oi != 0x7fffffff && (ai == 0x7fffffff || ov > av || (ov == av && oi < ai))) { av = ov; ai = oi; }
    }
    float sum = 0.f;
    for (int c = lane; c < G; c += 32) {
      const float* o = stat_part + ((size_t)c * MAX_M + r) * 4;
      const float cm = ldcg(o);
      if (cm != -INFINITY) sum += ldcg(o + 1) * expf(cm - mx);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) { rmax[r] = mx; rsum[r] = sum; rarg[r] = ai; }
  }
  named_sync(1, CONSUMER_THREADS);
}

__device__ __noinline__ float prob_of(float logit, float temperature, float rmax, float rsum) {
  return __fdiv_rn(expf(__fsub_rn(__fdiv_rn(logit, temperature), rmax)), rsum);
}

}  // namespace spd
