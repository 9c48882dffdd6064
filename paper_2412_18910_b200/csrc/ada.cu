// Host side of the C ABI declared in include/ada.h: argument checks, workspace carving, and the
// order in which the kernels of ada_kernels.cuh are enqueued for each step of Algorithm 1.
// Every step of the path runs in those kernels; nothing is computed on the host except the
// rotary table at initialisation.
#include "ada.h"

#include <cuda.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "ada_kernels.cuh"
#include "ada_pass.cuh"
#include "ada_gemm_tc.cuh"
#include "ada_attn_rows.cuh"

#include <unordered_map>
#include <utility>

using namespace ada;
typedef __nv_bfloat16 bf16;

namespace {

struct LayerW {
  const bf16 *wq, *wk, *wv, *wo, *wg, *wu, *wd, *na, *nm;
};

}  // namespace

struct ada_ctx {
  ada_config c;
  cudaStream_t stream;
  cudaStream_t capture_stream;  // private, only ever used to record the step graph (nothing executes on it)
  int B, TM;              // batch, rows of a decode pass of the multi-kernel path
  int pages_per_seq, n_pages;
  std::vector<LayerW> layers;
  LayerW eagle;
  const bf16 *embed, *lm_head, *final_norm, *eagle_fc, *ldlp_w1, *ldlp_b1, *ldlp_w2, *ldlp_b2, *ldlp_wr, *ldlp_br;
  // workspace pieces (device)
  bf16 *tk, *tv, *dk, *dv;          // KV pools: target [page][L][H][ps][hd], draft [page][1][H][ps][hd]
  int *page_table;                  // [B][pages_per_seq]
  float2 *rope;                     // [cap][hd/2]
  float *feat;                      // [B][cap][d]
  float *dfeat;                     // [B][nmax][d]
  int *tok;                         // [B][cap]
  SeqState *st;                     // [B]
  Counters *cnt;
  Pass *pass;
  float *h, *qkv, *ss_rows, *qrot, *attn_part, *gemm_part, *ldlp_h, *ldlp_h2, *ldlp_z, *dlp, *dfl, *dcum;
  bf16 *xhi, *xlo, *x2hi, *x2lo;    // [TP][ldx], [TP][ldx2]
  int ldx, ldx2;
  float4 *amax;
  int *draft, *target, *force_n_dev, *chunk_tok, *forced_buf;
  float2 *vtop, *dtop;
  const int *force_draft;           // user device pointer or null
  int has_force_n;
  int host_force_n[ADA_MAX_BATCH];
  size_t part_floats;
  // persistent pass kernel (batch 1): device copies of the layer pointer tables and its scratch
  int use_pass, n_sm;
  // tensor-core GEMM of the multi-row path (passes of up to 88 rows): tensor maps of every weight matrix and of
  // the activation planes, found by base pointer
  TensorMap128 *d_tcmaps;
  int n_tcmaps;
  std::unordered_map<const void *, int> tcmap_of, tcmap_wide_of;   // (wide: the planes in boxes of 128 rows)
  LayerPtrs *d_layers, *d_eagle;
  TensorMap128 *d_maps;
  int n_maps;
  float *ss_part, *attn_part2;
  bf16 *xa, *at, *ac, *fc;            // activation tiles (xstore layout), 2048 elements per 64 k
  int *attn_cnt;
  float4 *amax2;
  unsigned *gbar;
  unsigned long long *phase_ns;
  // bookkeeping
  long long launches;
  cudaGraphExec_t graph;
  int graph_launches;
  int graph_key;                    // configuration the graph was captured for
  int *out_acc, *out_emit, *out_nemit, *out_nused;   // internal outputs of ada_step
  // per-kernel timing for roofline reports (off by default): event pairs around GEMM / attention launches
  int prof;
  int pdl;                      // 1: the multi-row chain is launched with programmatic serialization (ADA_NO_PDL unset)
  std::vector<cudaEvent_t> ev_pool;
  struct ProfRec { int cls; int ev; double bytes; };
  std::vector<ProfRec> prof_recs;
  int ev_used;
  std::string err;
  int enqueue_failed;               // a helper could not enqueue part of a call (its text is in err)
};

namespace {

int fail(ada_ctx *ctx, int code, const char *msg) {
  if (ctx) ctx->err = msg;
  return code;
}

#define LAUNCH(ctx, kernel, grid, block, smem, ...)                         \
  do {                                                                      \
    kernel<<<grid, block, smem, (ctx)->stream>>>(__VA_ARGS__);              \
    (ctx)->launches++;                                                      \
  } while (0)

// Launch with the programmatic-serialization attribute: the kernel may begin while the kernel before it in the stream
// still runs and waits inside (pdl_wait) before it touches anything that kernel writes.  Only for kernels that wait in
// every thread before their first dependent access and before returning.
template <typename... KArgs, typename... Args>
void launch_pdl(ada_ctx *x, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args &&...args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = x->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = x->pdl;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
  x->launches++;
}

// Event pair around the launches made by `body` when profiling is on.
template <typename F>
void timed(ada_ctx *x, int cls, double bytes, F body) {
  if (!x->prof || x->ev_used + 2 > (int)x->ev_pool.size()) { body(); return; }
  const int e0 = x->ev_used;
  x->ev_used += 2;
  cudaEventRecord(x->ev_pool[e0], x->stream);
  body();
  cudaEventRecord(x->ev_pool[e0 + 1], x->stream);
  x->prof_recs.push_back({cls, e0, bytes});
}

struct Carver {
  char *base;
  size_t off;
  template <typename T>
  T *take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

bool config_ok(const ada_config *c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->n_layers > ADA_MAX_LAYERS) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_heads < 1 || c->d_model != c->n_heads * c->head_dim) return false;
  if (c->d_model > 1024 * kSsSegs) return false;   // the rows' sums of squares are kept per 1024-column segment
  if (c->d_model % 64 || c->d_ffn % 16 || c->d_ffn < 16 || c->vocab % 16 || c->vocab < 16) return false;
  if (c->ldlp_hidden < 1 || c->n_max < 1 || c->n_max > ADA_MAX_NMAX) return false;
  if (c->ldlp_mode != 0 && c->ldlp_mode != 1) return false;
  if (c->ddd_threshold < 0.f && c->max_batch != 1) return false;
  if (c->ldlp_mode == 1 && (c->ldlp_blocks < 0 || c->ldlp_blocks > 8 || c->k_min < 1 || c->k_min > c->n_max)) return false;
  if (c->max_batch < 1 || c->max_batch > ADA_MAX_BATCH) return false;
  if (c->max_batch * (c->n_max + 1) > 88) return false;
  // prompts and batches run the multi-row tensor-core GEMM, whose weight boxes are 128 rows high
  if (c->d_model < 128 || c->d_ffn < 128 || c->vocab < 128) return false;
  if (c->page_size != 64 || c->kv_capacity < 64 || c->kv_capacity % c->page_size) return false;
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 1.f)) return false;
  return true;
}

int rows_per_pass(const ada_config *c) {
  int t = c->max_batch * (c->n_max + 1);
  return t < 16 ? 16 : ((t + 7) / 8) * 8;
}

// K splits of the tensor-core GEMM: the smallest count that fills whole waves of one CTA per SM well (each split
// costs a round trip of partial sums), with at least four 64-k boxes per split.
int plan_tc_splits(int tiles, int K) {
  const int sms = 148;   // B200; the split is part of the arithmetic (summation order), so it follows the shape alone
  const int kboxes = (K + 63) / 64;
  // Cost of a launch relative to its weight bytes at full rate: how full the waves of one CTA per SM are, plus what
  // every further split adds in partial sums written and read back (128 rows x 4 bytes per output column against
  // 2 K bytes of weights, at about a third of the streaming rate).  Measured on the 7B shapes: gate-up (86 tiles,
  // K = 4096) is 8 % faster with 3 splits (1.7 waves) than with 5 (2.9 waves); O / down (16 tiles) are best at 8-9.
  const double per_split = 384.0 / (double)K;
  int best = 1;
  double best_cost = 1e30;
  for (int S = 1; S <= 16 && S * 4 <= (kboxes > 4 ? kboxes : 4); ++S) {
    const int ctas = tiles * S, waves = (ctas + sms - 1) / sms;
    const double cost = (double)waves * sms / ctas + per_split * (S - 1);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = S; }
  }
  return best;
}
int tc_tiles(int epi, int nseg, int Nseg) { return epi == EPI_SWIGLU ? (Nseg + 127) / 128 : nseg * ((Nseg + 255) / 256); }

size_t part_need_tc(int epi, int nseg, int Nseg, int K) {
  const int S = epi == EPI_ARGMAX ? 1 : plan_tc_splits(tc_tiles(epi, nseg, Nseg), K);
  const size_t Ntot = epi == EPI_SWIGLU ? 2 * (size_t)Nseg : (size_t)nseg * Nseg;
  return epi == EPI_ARGMAX ? 0 : (size_t)S * kTcRowsMax * Ntot;   // (every GEMM but the LM head leaves its sums here)
}

// Lays the workspace out; with base == nullptr only measures it.
size_t carve(ada_ctx *x, const ada_config *c, char *base) {
  Carver w{base, 0};
  const size_t d = c->d_model, F = c->d_ffn, V = c->vocab, L = c->n_layers, H = c->n_heads, hd = c->head_dim;
  const size_t B = c->max_batch, cap = c->kv_capacity, ps = c->page_size;
  const int TM = rows_per_pass(c);
  const size_t TP = kTcRowsMax;   // row scratch holds the largest pass of any engine: prompts go through 128-row chunks
  const size_t pps = cap / ps, pages = pps * B;
  x->B = (int)B; x->TM = TM; x->pages_per_seq = (int)pps; x->n_pages = (int)pages;
  x->tk = w.take<bf16>(pages * L * H * ps * hd);
  x->tv = w.take<bf16>(pages * L * H * ps * hd);
  x->dk = w.take<bf16>(pages * H * ps * hd);
  x->dv = w.take<bf16>(pages * H * ps * hd);
  x->page_table = w.take<int>(B * pps);
  x->rope = w.take<float2>(cap * (hd / 2));
  x->feat = w.take<float>(B * cap * d);
  x->dfeat = w.take<float>(B * c->n_max * d);
  x->tok = w.take<int>(B * cap);
  x->st = w.take<SeqState>(B);
  x->cnt = w.take<Counters>(1);
  x->pass = w.take<Pass>(1);
  x->h = w.take<float>(TP * d);
  x->qkv = w.take<float>(16 * 3 * d);   // the persistent pass kernel's q, k, v rows
  x->ss_rows = w.take<float>(TP * kSsSegs);
  x->qrot = w.take<float>(TP * d);
  x->attn_part = w.take<float>(H * kAttnSplits * (size_t)kMaxRows * (hd + 2));
  const size_t ldx = 2 * d, ldx2 = ((F + 63) / 64) * 64 > d ? ((F + 63) / 64) * 64 : d;
  x->ldx = (int)ldx; x->ldx2 = (int)ldx2;
  x->xhi = w.take<bf16>(TP * ldx);
  x->xlo = w.take<bf16>(TP * ldx);
  x->x2hi = w.take<bf16>(TP * ldx2);
  x->x2lo = w.take<bf16>(TP * ldx2);
  size_t pf = 0;
  auto upd = [&](size_t v) { if (v > pf) pf = v; };
  {
    upd(part_need_tc(EPI_STORE, 3, (int)d, (int)d));
    upd(part_need_tc(EPI_RESID, 1, (int)d, (int)d));
    upd(part_need_tc(EPI_SWIGLU, 1, (int)F, (int)d));
    upd(part_need_tc(EPI_RESID, 1, (int)d, (int)F));
    upd(part_need_tc(EPI_ARGMAX, 1, (int)V, (int)d));
    upd(part_need_tc(EPI_STORE, 1, (int)d, (int)(2 * d)));
  }
  x->part_floats = pf;
  x->gemm_part = w.take<float>(pf ? pf : 1);
  x->amax = w.take<float4>(((V + 255) / 256) * TP);
  x->ldlp_h = w.take<float>(B * c->ldlp_hidden);
  x->ldlp_h2 = w.take<float>(B * c->ldlp_hidden);
  x->ldlp_z = w.take<float>(B * 16);
  x->draft = w.take<int>(B * c->n_max);
  x->target = w.take<int>(B * (c->n_max + 1));
  x->force_n_dev = w.take<int>(B);
  x->forced_buf = w.take<int>(B * c->n_max);
  x->dlp = w.take<float>(B * c->n_max);
  x->dfl = w.take<float>(B * c->n_max);
  x->dcum = w.take<float>(B);
  x->chunk_tok = w.take<int>(kMaxRows);
  x->vtop = w.take<float2>(B * (c->n_max + 1) + kMaxRows);
  x->dtop = w.take<float2>(B * c->n_max + kMaxRows);
  x->out_acc = w.take<int>(B);
  x->out_emit = w.take<int>(B * (c->n_max + 1));
  x->out_nemit = w.take<int>(B);
  x->out_nused = w.take<int>(B);
  x->d_layers = w.take<LayerPtrs>(L);
  x->d_eagle = w.take<LayerPtrs>(1);
  x->n_maps = (int)(7 * (L + 1) + 2 + 8);
  x->d_maps = w.take<TensorMap128>(x->n_maps);
  x->n_tcmaps = (int)(7 * (L + 1) + 2 + 8);
  x->d_tcmaps = w.take<TensorMap128>(x->n_tcmaps);
  x->xa = w.take<bf16>(((d + 63) / 64) * 2048);
  x->at = w.take<bf16>(((d + 63) / 64) * 2048);
  x->ac = w.take<bf16>(((F + 63) / 64) * 2048);
  x->fc = w.take<bf16>(((2 * d + 63) / 64) * 2048);
  x->ss_part = w.take<float>(256 * 16);
  x->attn_part2 = w.take<float>(H * kPassMaxSplits * 16 * (hd + 2));
  x->attn_cnt = w.take<int>(H);
  x->amax2 = w.take<float4>(256 * 16);
  x->gbar = w.take<unsigned>(64);
  x->phase_ns = w.take<unsigned long long>(512 + 4 * 512);
  return (w.off + 255) & ~(size_t)255;
}

// What follows a GEMM's sums (the reduction kernel launched after it).
struct Reduce {
  enum Kind { QKV_ROPE, H, SWIGLU, NONE } kind;
  // H: residual add or plain store, and the norm whose input planes are written (null: none)
  int resid; const bf16 *gain;
  // QKV_ROPE: the cache the rows go to
  bf16 *kpool, *vpool; int L, layer;
};

// Sums of X W^T into the scratch buffer (tensor-core GEMM, K splits), then the reduction kernel `r`; the LM head
// (EPI_ARGMAX, r.kind NONE) reduces the greedy choice itself.  W0..W2: row segments (STORE) or gate/up (SWIGLU).
// False (with the context's error text set) if an operand has no tensor map; every operand of the path is registered
// at initialisation.
bool gemm(ada_ctx *x, int epi, const bf16 *W0, const bf16 *W1, const bf16 *W2, int nseg, int Nseg, int K,
          const bf16 *Xhi, const bf16 *Xlo, const Reduce &r, float *logits, int use_lm_rows) {
  const ada_config &c = x->c;
  GemmTcArgs t;
  memset(&t, 0, sizeof(t));
  const bf16 *Ws[3] = {W0, W1, W2};
  const bool wide = x->TM > kTcRows;   // a prompt chunk: planes in boxes of 128 rows
  auto map_of = [&](const void *base) -> const TensorMap128 * {
    auto it = x->tcmap_of.find(base);
    return it == x->tcmap_of.end() ? nullptr : x->d_tcmaps + it->second;
  };
  auto plane_of = [&](const void *base) -> const TensorMap128 * {
    if (!wide) return map_of(base);
    auto it = x->tcmap_wide_of.find(base);
    return it == x->tcmap_wide_of.end() ? nullptr : x->d_tcmaps + it->second;
  };
  for (int i = 0; i < 3; ++i)
    if (Ws[i]) t.wmap[i] = map_of(Ws[i]);
  t.xhi_map = plane_of(Xhi);
  t.xlo_map = plane_of(Xlo);
  if (!t.wmap[0] || (W1 && !t.wmap[1]) || (W2 && !t.wmap[2]) || !t.xhi_map || !t.xlo_map) {
    x->err = "gemm: operand without a tensor map";
    x->enqueue_failed = 1;
    return false;
  }
  t.epi = epi; t.nseg = nseg; t.Nseg = Nseg; t.K = K;
  const int tiles = tc_tiles(epi, nseg, Nseg);
  t.S = epi == EPI_ARGMAX ? 1 : plan_tc_splits(tiles, K);
  t.to_part = epi != EPI_ARGMAX;
  t.part = x->gemm_part;
  t.logits = logits; t.ldl = c.vocab; t.amax = x->amax;
  t.pass = x->pass; t.use_lm_rows = use_lm_rows; t.cnts = x->cnt;
  const int rows = wide ? kTcRowsMax : kTcRows;
  const int d = c.d_model;
  const double wb = 2.0 * (double)Nseg * (double)K * (epi == EPI_SWIGLU ? 2 : nseg);
  timed(x, 0, wb, [&] {
    if (wide) launch_pdl(x, k_gemm_tc<kTcRowsMax>, dim3(tiles, t.S), kTcThreads, TcShape<kTcRowsMax>::kSmemBytes, t);
    else launch_pdl(x, k_gemm_tc<kTcRows>, dim3(tiles, t.S), kTcThreads, TcShape<kTcRows>::kSmemBytes, t);
    if (r.kind == Reduce::H) {
      ReduceHArgs a;
      a.part = x->gemm_part; a.S = t.S; a.Ntot = Nseg; a.h = x->h; a.d = d; a.resid = r.resid; a.gain = r.gain;
      a.xhi = x->xhi; a.xlo = x->xlo; a.ldx = x->ldx; a.ss_part = x->ss_rows; a.pass = x->pass;
      launch_pdl(x, k_reduce_h, dim3((d + 1023) / 1024, rows), 256, 0, a);
    } else if (r.kind == Reduce::QKV_ROPE) {
      ReduceQkvArgs a;
      a.part = x->gemm_part; a.S = t.S; a.ss_part = x->ss_rows; a.eps = c.rms_eps; a.rope = x->rope; a.qout = x->qrot;
      a.kpool = r.kpool; a.vpool = r.vpool; a.page_table = x->page_table; a.pages_per_seq = x->pages_per_seq;
      a.page_size = c.page_size; a.L = r.L; a.layer = r.layer; a.H = c.n_heads; a.hd = c.head_dim;
      a.qscale = 1.0f / sqrtf((float)c.head_dim); a.pass = x->pass;
      launch_pdl(x, k_reduce_qkv, dim3((c.n_heads * (c.head_dim / 2) + 255) / 256, rows), 256, 0, a);
    } else if (r.kind == Reduce::SWIGLU) {
      ReduceSwigluArgs a;
      a.part = x->gemm_part; a.S = t.S; a.F = Nseg; a.ss_part = x->ss_rows; a.eps = c.rms_eps; a.d = d;
      a.ohi = x->x2hi; a.olo = x->x2lo; a.ldo = x->ldx2; a.pass = x->pass;
      const int blocks = (rows * (Nseg / 4) + 255) / 256;
      launch_pdl(x, k_reduce_swiglu, dim3(blocks < 1184 ? blocks : 1184), 256, 0, a);
    }
  });
  return true;
}

void attention(ada_ctx *x, bf16 *kpool, bf16 *vpool, int L, int layer) {
  const ada_config &c = x->c;
  // Query rows of a sequence in groups across grid.z.  A prompt chunk is one sequence with up to 128 rows (whatever the
  // batch size of the engine): groups of 16 rows.  Decode passes have at most n_max + 1 rows per sequence: groups of 8
  // rows whose hi and lo halves share one 16-row tile (half the products per key); every decode row of a sequence goes
  // through this form, whatever the shape of its pass.
  const bool wide = x->TM > kTcRows;
  const int nrg = wide ? (x->TM + kRowGroup - 1) / kRowGroup : (x->TM / x->B + 7) / 8;
  dim3 g1(c.n_heads, kAttnSplits, x->B * nrg);
  dim3 g2(c.n_heads, x->TM);
  auto rows_kernel = [&](auto kernel, int smem) {
    launch_pdl(x, kernel, g1, dim3(128), (size_t)smem, x->pass, x->qrot, kpool, vpool, x->page_table, x->pages_per_seq,
               c.page_size, L, layer, c.n_heads, x->attn_part, nrg, c.kv_capacity, x->cnt);
  };
  timed(x, 1, 0.0, [&] {
    if (c.head_dim == 128) {
      if (wide) rows_kernel(k_attn_rows<128, false>, attn_rows_smem_bytes<128>());
      else rows_kernel(k_attn_rows<128, true>, attn_rows_smem_bytes<128>());
      launch_pdl(x, k_attn_combine<128>, g2, 128, 0, x->pass, x->attn_part, x->xhi, x->xlo, x->ldx, c.kv_capacity);
    } else {
      if (wide) rows_kernel(k_attn_rows<64, false>, attn_rows_smem_bytes<64>());
      else rows_kernel(k_attn_rows<64, true>, attn_rows_smem_bytes<64>());
      launch_pdl(x, k_attn_combine<64>, g2, 64, 0, x->pass, x->attn_part, x->xhi, x->xlo, x->ldx, c.kv_capacity);
    }
  });
}

// One pre-norm decoder block over the rows of x->pass.  On entry the residual stream is in x->h, the planes hold
// split(h * norm_attn gain) and the rows' sums of squares are in x->ss_rows (written by whatever produced h); on exit
// the same holds for `next_gain`, the norm that follows the block (null: none, planes are left alone).
void decoder_block(ada_ctx *x, const LayerW &w, bf16 *kpool, bf16 *vpool, int L, int layer, const bf16 *next_gain) {
  const ada_config &c = x->c;
  const int d = c.d_model, F = c.d_ffn;
  Reduce qkv{Reduce::QKV_ROPE, 0, nullptr, kpool, vpool, L, layer};
  gemm(x, EPI_STORE, w.wq, w.wk, w.wv, 3, d, d, x->xhi, x->xlo, qkv, nullptr, 0);
  attention(x, kpool, vpool, L, layer);
  Reduce o{Reduce::H, 1, w.nm, nullptr, nullptr, 0, 0};
  gemm(x, EPI_RESID, w.wo, nullptr, nullptr, 1, d, d, x->xhi, x->xlo, o, nullptr, 0);
  Reduce sw{Reduce::SWIGLU, 0, nullptr, nullptr, nullptr, 0, 0};
  gemm(x, EPI_SWIGLU, w.wg, w.wu, nullptr, 1, F, d, x->xhi, x->xlo, sw, nullptr, 0);
  Reduce down{Reduce::H, 1, next_gain, nullptr, nullptr, 0, 0};
  gemm(x, EPI_RESID, w.wd, nullptr, nullptr, 1, d, F, x->x2hi, x->x2lo, down, nullptr, 0);
}

// Target over the rows of x->pass: embedding, all layers, final norm (features kept per position).
void target_rows(ada_ctx *x) {
  const ada_config &c = x->c;
  LAUNCH(x, k_embed, x->TM, 256, 0, x->pass, x->embed, x->h, c.d_model, x->layers[0].na, x->xhi, x->xlo, x->ldx, x->ss_rows,
         kSsSegs);
  for (int l = 0; l < c.n_layers; ++l)
    decoder_block(x, x->layers[l], x->tk, x->tv, c.n_layers, l, l + 1 < c.n_layers ? x->layers[l + 1].na : nullptr);
  LAUNCH(x, k_rmsnorm, x->TM, 256, 0, x->pass, x->h, x->final_norm, c.rms_eps, c.d_model, x->xhi, x->xlo, x->ldx,
         x->feat, c.kv_capacity);
}

// Shared LM head + greedy choice over the rows staged in (xhi, xlo).
void lm_head(ada_ctx *x, const bf16 *Xhi, const bf16 *Xlo, int use_lm_rows, int *tok_out, float2 *top_out,
             const int *forced, float *logits) {
  const ada_config &c = x->c;
  Reduce none{Reduce::NONE, 0, nullptr, nullptr, nullptr, 0, 0};
  gemm(x, EPI_ARGMAX, x->lm_head, nullptr, nullptr, 1, c.vocab, c.d_model, Xhi, Xlo, none, logits, use_lm_rows);
  LAUNCH(x, k_argmax_final, x->TM, 32, 0, x->amax, (c.vocab + 255) / 256, kTcRowsMax, x->pass, use_lm_rows, tok_out, top_out,
         forced);
}

// Draft head over the rows of x->pass (already built for `step`).
void draft_rows(ada_ctx *x, int step, bool with_lm) {
  const ada_config &c = x->c;
  const int d = c.d_model;
  LAUNCH(x, k_eagle_input, x->TM, 256, 0, x->pass, x->embed, x->feat, c.kv_capacity, x->dfeat, c.n_max, step, d, x->xhi,
         x->xlo, x->ldx);
  Reduce fc{Reduce::H, 0, x->eagle.na, nullptr, nullptr, 0, 0};   // h = fc([e ; f]), planes for the head's layer
  gemm(x, EPI_STORE, x->eagle_fc, nullptr, nullptr, 1, d, 2 * d, x->xhi, x->xlo, fc, nullptr, 0);
  decoder_block(x, x->eagle, x->dk, x->dv, 1, 0, nullptr);
  if (with_lm) {
    LAUNCH(x, k_split_lm_rows, x->B, 256, 0, x->pass, x->h, d, x->x2hi, x->x2lo, x->ldx2, x->dfeat, c.n_max, step);
    lm_head(x, x->x2hi, x->x2lo, 1, x->draft, x->dtop, x->force_draft, nullptr);
  }
}

// 2-D bf16 tensor map over a row-major [rows][cols] matrix: box = 64 columns x box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_map(EncodeTiledFn fn, TensorMap128 *out, const void *base, size_t rows, size_t cols, unsigned box_rows) {
  static_assert(sizeof(CUtensorMap) == sizeof(TensorMap128), "tensor map size");
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// All tensor maps of a context, in the order ada_pass.cuh documents.
bool build_maps(ada_ctx *x, std::vector<TensorMap128> &maps) {
  void *sym = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym) return false;
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(sym);
  const ada_config &c = x->c;
  const size_t d = c.d_model, F = c.d_ffn, V = c.vocab;
  maps.assign(x->n_maps, TensorMap128());
  bool ok = true;
  // box height of each matrix = rows of one m tile of its slabs (same arithmetic as the kernel's make_slab)
  const unsigned b_qkv = slab_box_rows(slab_rpc((int)d, 3, x->n_sm), false);
  // matrices with d output rows may be cut along K too (see make_slab): their slabs are then taller
  auto d_rows = [&](size_t K) {
    const int ks = slab_ksplit((int)d, (int)K, x->n_sm);
    const int groups = ks > 1 ? x->n_sm / ks : x->n_sm;
    return (unsigned)slab_box_rows(((int)d + groups - 1) / groups, false);
  };
  const unsigned b_wo = d_rows(d), b_wd = d_rows(F), b_fc = d_rows(2 * d);
  const unsigned b_f = slab_box_rows(slab_rpc((int)F, 1, x->n_sm), true);
  const unsigned b_v = slab_box_rows(slab_rpc((int)V, 1, x->n_sm), false);
  auto layer = [&](int base, const LayerW &a) {
    ok = ok && encode_map(fn, &maps[base + MAP_WQ], a.wq, d, d, b_qkv) && encode_map(fn, &maps[base + MAP_WK], a.wk, d, d, b_qkv) &&
         encode_map(fn, &maps[base + MAP_WV], a.wv, d, d, b_qkv) && encode_map(fn, &maps[base + MAP_WO], a.wo, d, d, b_wo) &&
         encode_map(fn, &maps[base + MAP_WG], a.wg, F, d, b_f) && encode_map(fn, &maps[base + MAP_WU], a.wu, F, d, b_f) &&
         encode_map(fn, &maps[base + MAP_WD], a.wd, d, F, b_wd);
  };
  for (int l = 0; l < c.n_layers; ++l) layer(7 * l, x->layers[l]);
  layer(7 * c.n_layers, x->eagle);
  const int m0 = 7 * (c.n_layers + 1);
  ok = ok && encode_map(fn, &maps[m0], x->eagle_fc, d, 2 * d, b_fc) && encode_map(fn, &maps[m0 + 1], x->lm_head, V, d, b_v);
  return ok;
}

// Tensor maps of the multi-row tensor-core GEMM: every weight matrix with a box of 64 k x 128 rows, the four
// activation planes with a box of 64 k x 88 rows; tcmap_of finds a map by the base pointer of its tensor.
bool build_tc_maps(ada_ctx *x, std::vector<TensorMap128> &maps) {
  void *sym = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym) return false;
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(sym);
  const ada_config &c = x->c;
  const size_t d = c.d_model, F = c.d_ffn, V = c.vocab;
  maps.assign(x->n_tcmaps, TensorMap128());
  x->tcmap_of.clear();
  bool ok = true;
  int next = 0;
  auto add = [&](const void *base, size_t rows, size_t cols, unsigned box_rows) {
    if (x->tcmap_of.count(base)) return;   // a tensor is looked up by its base pointer
    ok = ok && next < x->n_tcmaps && encode_map(fn, &maps[next], base, rows, cols, box_rows);
    x->tcmap_of[base] = next++;
  };
  auto layer = [&](const LayerW &a) {
    add(a.wq, d, d, 128); add(a.wk, d, d, 128); add(a.wv, d, d, 128); add(a.wo, d, d, 128);
    add(a.wg, F, d, 128); add(a.wu, F, d, 128); add(a.wd, d, F, 128);
  };
  for (int l = 0; l < c.n_layers; ++l) layer(x->layers[l]);
  layer(x->eagle);
  add(x->eagle_fc, d, 2 * d, 128);
  add(x->lm_head, V, d, 128);
  add(x->xhi, kTcRowsMax, x->ldx, kTcRows); add(x->xlo, kTcRowsMax, x->ldx, kTcRows);
  add(x->x2hi, kTcRowsMax, x->ldx2, kTcRows); add(x->x2lo, kTcRowsMax, x->ldx2, kTcRows);
  x->tcmap_wide_of.clear();
  auto add_wide = [&](const void *base, size_t cols) {
    ok = ok && next < x->n_tcmaps && encode_map(fn, &maps[next], base, kTcRowsMax, cols, kTcRowsMax);
    x->tcmap_wide_of[base] = next++;
  };
  add_wide(x->xhi, x->ldx); add_wide(x->xlo, x->ldx); add_wide(x->x2hi, x->ldx2); add_wide(x->x2lo, x->ldx2);
  return ok;
}

// Bytes of weights one pass streams (each once): for the per-launch roofline record.
double pass_weight_bytes(const ada_ctx *x, int mode, int with_lm) {
  const ada_config &c = x->c;
  const double d = c.d_model, F = c.d_ffn, V = c.vocab;
  const double layer = 4 * d * d + 3 * d * F;
  double p = mode == 0 ? c.n_layers * layer : 2 * d * d + layer;
  if (with_lm) p += V * d;
  return 2.0 * p;
}

// One persistent launch for a whole pass over the rows of x->pass (at most 16 rows, one sequence).
// mode 0: target (embedding, layers, final norm -> features, LM head -> target choices)
// mode 1: draft head (fc on [e ; f], its layer, optionally the LM head on the last rows)
void run_pass(ada_ctx *x, int mode, int step, int with_lm, float *logits, int *tok_out, float2 *top_out,
              const int *forced) {
  const ada_config &c = x->c;
  PassParams p;
  memset(&p, 0, sizeof(p));
  p.pass = x->pass;
  p.layers = mode == 0 ? x->d_layers : x->d_eagle;
  p.maps = x->d_maps;
  p.map_layer0 = mode == 0 ? 0 : 7 * c.n_layers;
  p.map_fc = 7 * (c.n_layers + 1); p.map_lm = p.map_fc + 1; p.map_planes = p.map_fc + 2;
  p.n_layers = mode == 0 ? c.n_layers : 1;
  p.cache_layers = p.n_layers;
  p.d = c.d_model; p.H = c.n_heads; p.hd = c.head_dim; p.F = c.d_ffn; p.V = c.vocab; p.eps = c.rms_eps;
  p.embed = x->embed; p.lm_head = x->lm_head; p.final_norm = x->final_norm; p.eagle_fc = x->eagle_fc;
  p.mode = mode; p.draft_step = step; p.with_lm = with_lm;
  p.h = x->h; p.qkv = x->qkv; p.ss_part = x->ss_part;
  p.xa = x->xa; p.at = x->at; p.ac = x->ac; p.fc = x->fc;
  p.feat = x->feat; p.cap = c.kv_capacity; p.dfeat = x->dfeat; p.nmax = c.n_max;
  p.rope = x->rope;
  p.kpool = mode == 0 ? x->tk : x->dk; p.vpool = mode == 0 ? x->tv : x->dv;
  p.page_table = x->page_table; p.pages_per_seq = x->pages_per_seq; p.page_size = c.page_size;
  p.attn_part = x->attn_part2; p.attn_cnt = x->attn_cnt;
  p.amax = x->amax2; p.logits = logits; p.tok_out = tok_out; p.top_out = top_out; p.forced = forced;
  p.gbar = x->gbar; p.cnt = x->cnt;
  p.lp_out = (mode == 1 && with_lm && x->c.ddd_threshold < 0.f) ? x->dlp : nullptr; p.tok_logit = x->dfl;
  p.phase_ns = (x->prof && mode == 0) ? x->phase_ns : nullptr;
  timed(x, 0, pass_weight_bytes(x, mode, with_lm), [&] {
    cudaMemsetAsync(x->gbar, 0, sizeof(unsigned), x->stream);
    // cooperative (all CTAs resident: they meet at grid barriers) in clusters of two (K-split pairs)
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(x->n_sm); lc.blockDim = dim3(kPassThreads); lc.dynamicSmemBytes = kPassSmemBytes; lc.stream = x->stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative; at[1].val.cooperative = 1;
    // ADA_PASS_NONCOOP=1 drops the cooperative attribute (same kernel, grid and clusters): Nsight Compute refuses
    // the launch with both attributes.  Residency of all clusters was checked at initialisation, and every
    // wait in the kernel is bounded, so without the attribute a grid that is not resident ends with a status
    // bit instead of the launch error.
    static const bool noncoop = getenv("ADA_PASS_NONCOOP") != nullptr;
    lc.attrs = at; lc.numAttrs = noncoop ? 1 : 2;
    cudaLaunchKernelEx(&lc, k_pass, p);
    x->launches++;
  });
}

void enqueue_ldlp(ada_ctx *x, int *d_n) {
  const ada_config &c = x->c;
  dim3 g((c.ldlp_hidden + 7) / 8, x->B), g4((c.ldlp_hidden + 3) / 4, x->B);
  LAUNCH(x, k_ldlp_hidden, g4, 128, 0, x->st, x->tok, x->feat, c.kv_capacity, x->embed, x->ldlp_w1, x->ldlp_b1,
         c.d_model, c.ldlp_hidden, x->ldlp_h);
  float *hin = x->ldlp_h, *hout = x->ldlp_h2;
  if (c.ldlp_mode == 1)
    for (int blk = 0; blk < c.ldlp_blocks; ++blk) {   // residual blocks of the scalar form, ping-pong buffers
      LAUNCH(x, k_ldlp_block, g, 256, 0, x->st, hin, hout, x->ldlp_wr + (size_t)blk * c.ldlp_hidden * c.ldlp_hidden,
             x->ldlp_br + (size_t)blk * c.ldlp_hidden, c.ldlp_hidden);
      float *t = hin; hin = hout; hout = t;
    }
  LAUNCH(x, k_ldlp_out, x->B, 512, 0, x->st, hin, x->ldlp_w2, x->ldlp_b2, c.ldlp_hidden, c.n_max, c.ldlp_mode, c.k_min,
         c.kv_capacity, x->force_n_dev, x->has_force_n, x->ldlp_z, d_n, x->cnt);
}

void enqueue_draft(ada_ctx *x) {
  const ada_config &c = x->c;
  for (int step = 0; step < c.n_max; ++step) {
    LAUNCH(x, k_rows_draft, 1, 32, 0, x->pass, x->st, x->tok, c.kv_capacity, x->draft, c.n_max, x->B, step, x->TM,
           x->cnt);
    if (x->use_pass) run_pass(x, 1, step, 1, nullptr, x->draft, x->dtop, x->force_draft);
    else draft_rows(x, step, true);
    if (c.ddd_threshold < 0.f)   // Section 4: the draft may grow past the predicted length
      LAUNCH(x, k_ddd_update, 1, 32, 0, x->st, x->dlp, x->dcum, c.ddd_threshold, c.n_max, c.kv_capacity, x->B, step);
  }
}

void enqueue_verify(ada_ctx *x, int only_seq, float *d_logits) {
  const ada_config &c = x->c;
  LAUNCH(x, k_rows_verify, 1, 32, 0, x->pass, x->st, x->tok, c.kv_capacity, x->draft, c.n_max, x->B, only_seq);
  if (x->use_pass) {
    run_pass(x, 0, 0, 1, d_logits, x->target, x->vtop, nullptr);
  } else {
    target_rows(x);
    lm_head(x, x->xhi, x->xlo, 0, x->target, x->vtop, nullptr, d_logits);
  }
}

// Multi-row passes over committed positions of one sequence, 128 rows per chunk: the target over positions
// [p_begin, p_end) (cache rows and features), the draft head over those of them below d_end (each needs the token after
// its position).  with_choice: the greedy choice after position p_end - 1 goes to chunk_tok.  chunk: the sequence's
// attention split size.  Returns the rows of the last chunk.
int enqueue_chunks(ada_ctx *x, int seq, int p_begin, int p_end, int d_end, bool with_choice, int chunk) {
  const ada_config &c = x->c;
  int last_rows = 0;
  const int TM0 = x->TM;
  x->TM = kTcRowsMax;
  for (int p0 = p_begin; p0 < p_end; p0 += x->TM) {
    const int R = (p_end - p0 < x->TM) ? p_end - p0 : x->TM;
    LAUNCH(x, k_rows_chunk, 1, 32, 0, x->pass, x->tok, c.kv_capacity, seq, p0, R, 0, x->B, chunk);
    target_rows(x);
    if (p0 + R == p_end) {  // the chunk that holds the last position: greedy choice after it
      if (with_choice) lm_head(x, x->xhi, x->xlo, 0, x->chunk_tok, x->vtop + x->B * (c.n_max + 1), nullptr, nullptr);
      last_rows = R;
    }
    const int Rd = (p0 + R <= d_end) ? R : (d_end - p0);
    if (Rd > 0) {
      LAUNCH(x, k_rows_chunk, 1, 32, 0, x->pass, x->tok, c.kv_capacity, seq, p0, Rd, 1, x->B, chunk);
      draft_rows(x, 0, false);
    }
  }
  x->TM = TM0;
  return last_rows;
}

// Status of an API call after its launches: ADA_ERR_STATE if a helper refused to enqueue part of it, ADA_ERR_CUDA if
// a launch failed, else ADA_OK.
int finish(ada_ctx *x, const char *what) {
  if (x->enqueue_failed) {
    x->enqueue_failed = 0;
    cudaGetLastError();
    return ADA_ERR_STATE;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    x->err = std::string(what) + ": " + cudaGetErrorString(e);
    return ADA_ERR_CUDA;
  }
  return ADA_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------------

extern "C" size_t ada_workspace_bytes(const ada_config *cfg) {
  if (!config_ok(cfg)) return 0;
  ada_ctx tmp;
  return carve(&tmp, cfg, nullptr);
}

extern "C" int ada_init(ada_ctx **out, const ada_config *cfg, const ada_weights *w, void *d_workspace,
                        size_t workspace_bytes, void *cuda_stream) {
  if (!out || !cfg || !w || !d_workspace) return ADA_ERR_NULL;
  if (!config_ok(cfg)) return ADA_ERR_BAD_CONFIG;
  if (((uintptr_t)d_workspace & 255) != 0) return ADA_ERR_WORKSPACE;
  const void *singles[] = {w->embed, w->lm_head, w->final_norm, w->eagle_fc, w->e_wq, w->e_wk, w->e_wv, w->e_wo,
                           w->e_gate, w->e_up, w->e_down, w->e_norm_attn, w->e_norm_mlp, w->ldlp_w1, w->ldlp_b1,
                           w->ldlp_w2, w->ldlp_b2};
  for (const void *p : singles)
    if (!p || ((uintptr_t)p & 15)) return ADA_ERR_NULL;
  if (cfg->ldlp_mode == 1 && cfg->ldlp_blocks > 0 && (!w->ldlp_wr || !w->ldlp_br)) return ADA_ERR_NULL;
  const void *const *per[] = {w->wq, w->wk, w->wv, w->wo, w->w_gate, w->w_up, w->w_down, w->norm_attn, w->norm_mlp};
  for (auto arr : per) {
    if (!arr) return ADA_ERR_NULL;
    for (int l = 0; l < cfg->n_layers; ++l)
      if (!arr[l] || ((uintptr_t)arr[l] & 15)) return ADA_ERR_NULL;
  }
  ada_ctx *x = new ada_ctx();
  x->c = *cfg;
  x->stream = (cudaStream_t)cuda_stream;
  const size_t need = carve(x, cfg, (char *)d_workspace);
  if (workspace_bytes < need) {
    delete x;
    return ADA_ERR_WORKSPACE;
  }
  x->layers.resize(cfg->n_layers);
  for (int l = 0; l < cfg->n_layers; ++l)
    x->layers[l] = LayerW{(const bf16 *)w->wq[l], (const bf16 *)w->wk[l], (const bf16 *)w->wv[l], (const bf16 *)w->wo[l],
                          (const bf16 *)w->w_gate[l], (const bf16 *)w->w_up[l], (const bf16 *)w->w_down[l],
                          (const bf16 *)w->norm_attn[l], (const bf16 *)w->norm_mlp[l]};
  x->eagle = LayerW{(const bf16 *)w->e_wq, (const bf16 *)w->e_wk, (const bf16 *)w->e_wv, (const bf16 *)w->e_wo,
                    (const bf16 *)w->e_gate, (const bf16 *)w->e_up, (const bf16 *)w->e_down,
                    (const bf16 *)w->e_norm_attn, (const bf16 *)w->e_norm_mlp};
  x->embed = (const bf16 *)w->embed; x->lm_head = (const bf16 *)w->lm_head; x->final_norm = (const bf16 *)w->final_norm;
  x->eagle_fc = (const bf16 *)w->eagle_fc;
  x->ldlp_w1 = (const bf16 *)w->ldlp_w1; x->ldlp_b1 = (const bf16 *)w->ldlp_b1;
  x->ldlp_w2 = (const bf16 *)w->ldlp_w2; x->ldlp_b2 = (const bf16 *)w->ldlp_b2;
  x->ldlp_wr = (const bf16 *)w->ldlp_wr; x->ldlp_br = (const bf16 *)w->ldlp_br;
  x->force_draft = nullptr; x->has_force_n = 0; x->launches = 0; x->graph = nullptr; x->graph_launches = 0;
  x->graph_key = -1;
  x->capture_stream = nullptr;
  x->prof = 0; x->ev_used = 0; x->enqueue_failed = 0;
  x->pdl = getenv("ADA_NO_PDL") ? 0 : 1;

  // rotary table: angle = pos * theta^(-2i/hd), evaluated in double, stored as (cos, sin) floats
  const int half = cfg->head_dim / 2, cap = cfg->kv_capacity;
  std::vector<float2> rope((size_t)cap * half);
  for (int i = 0; i < half; ++i) {
    const double inv = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)cfg->head_dim);
    for (int p = 0; p < cap; ++p) {
      const double ang = (double)p * inv;
      rope[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
    }
  }
  // page table: page i of sequence b is pool page i*B + b (sequences interleaved in the pool)
  std::vector<int> pt((size_t)x->B * x->pages_per_seq);
  for (int b = 0; b < x->B; ++b)
    for (int i = 0; i < x->pages_per_seq; ++i) pt[(size_t)b * x->pages_per_seq + i] = i * x->B + b;
  cudaError_t e = cudaMemcpyAsync(x->rope, rope.data(), rope.size() * sizeof(float2), cudaMemcpyHostToDevice, x->stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(x->page_table, pt.data(), pt.size() * sizeof(int), cudaMemcpyHostToDevice, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->st, 0, sizeof(SeqState) * x->B, x->stream);
  // cache rows start finite (zero): the attention kernels copy whole blocks, and a masked key still multiplies its value row by 0
  {
    const size_t pool = (size_t)x->n_pages * cfg->n_heads * cfg->page_size * cfg->head_dim * sizeof(bf16);
    if (e == cudaSuccess) e = cudaMemsetAsync(x->tk, 0, pool * cfg->n_layers, x->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(x->tv, 0, pool * cfg->n_layers, x->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(x->dk, 0, pool, x->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(x->dv, 0, pool, x->stream);
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(x->cnt, 0, sizeof(Counters), x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->pass, 0, sizeof(Pass), x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->tok, 0, sizeof(int) * (size_t)x->B * cap, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->draft, 0, sizeof(int) * x->B * cfg->n_max, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->target, 0, sizeof(int) * x->B * (cfg->n_max + 1), x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->force_n_dev, 0, sizeof(int) * x->B, x->stream);
  // activation staging rows beyond the live ones are read by the tensor-core tiles: keep them finite
  if (e == cudaSuccess) e = cudaMemsetAsync(x->xhi, 0, sizeof(bf16) * (size_t)kTcRowsMax * x->ldx, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->xlo, 0, sizeof(bf16) * (size_t)kTcRowsMax * x->ldx, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->x2hi, 0, sizeof(bf16) * (size_t)kTcRowsMax * x->ldx2, x->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->x2lo, 0, sizeof(bf16) * (size_t)kTcRowsMax * x->ldx2, x->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(x->stream);  // host vectors go out of scope
  // persistent pass kernel: one sequence, at most 16 rows per pass (its attention phase reads one sequence's cache)
  x->use_pass = 0;
  if (e == cudaSuccess && cfg->max_batch == 1 && x->TM <= 16) {
    int dev = 0, sms = 0, per_sm = 0;
    e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_pass, cudaFuncAttributeMaxDynamicSharedMemorySize, kPassSmemBytes);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pass, kPassThreads, kPassSmemBytes);
    // slabs must fit the tensor-memory accumulators: one m tile (128 rows) for gate/up, two otherwise
    const bool fits = sms >= 4 && slab_rpc(cfg->d_ffn, 1, sms) <= 128 && slab_rpc(cfg->vocab, 1, sms) <= 256 &&
                      slab_rpc(cfg->d_model, 3, sms) <= 256;
    // the kernel runs as clusters of two CTAs, one CTA per SM: an even grid, all clusters resident at once
    const int grid = sms & ~1;
    int max_clusters = 0;
    if (e == cudaSuccess && per_sm >= 1) {
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(grid); lc.blockDim = dim3(kPassThreads); lc.dynamicSmemBytes = kPassSmemBytes;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at; lc.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&max_clusters, k_pass, &lc) != cudaSuccess) { max_clusters = 0; cudaGetLastError(); }
    }
    if (e == cudaSuccess && per_sm >= 1 && sms <= 256 && fits && max_clusters >= grid / 2) {
      x->use_pass = 1;
      x->n_sm = grid;
      std::vector<LayerPtrs> lp(cfg->n_layers);
      for (int l = 0; l < cfg->n_layers; ++l) {
        const LayerW &a = x->layers[l];
        lp[l] = LayerPtrs{a.wq, a.wk, a.wv, a.wo, a.wg, a.wu, a.wd, a.na, a.nm};
      }
      const LayerW &a = x->eagle;
      LayerPtrs ep{a.wq, a.wk, a.wv, a.wo, a.wg, a.wu, a.wd, a.na, a.nm};
      e = cudaMemcpy(x->d_layers, lp.data(), sizeof(LayerPtrs) * lp.size(), cudaMemcpyHostToDevice);
      if (e == cudaSuccess) e = cudaMemcpy(x->d_eagle, &ep, sizeof(LayerPtrs), cudaMemcpyHostToDevice);
      std::vector<TensorMap128> maps;
      if (e == cudaSuccess && !build_maps(x, maps)) e = cudaErrorUnknown;
      if (e == cudaSuccess) e = cudaMemcpy(x->d_maps, maps.data(), sizeof(TensorMap128) * maps.size(), cudaMemcpyHostToDevice);
      // planes start finite: rows past the live ones are read by the tensor-core tiles
      const size_t dd = cfg->d_model, FF = cfg->d_ffn;
      if (e == cudaSuccess) e = cudaMemset(x->xa, 0, ((dd + 63) / 64) * 4096);
      if (e == cudaSuccess) e = cudaMemset(x->at, 0, ((dd + 63) / 64) * 4096);
      if (e == cudaSuccess) e = cudaMemset(x->ac, 0, ((FF + 63) / 64) * 4096);
      if (e == cudaSuccess) e = cudaMemset(x->fc, 0, ((2 * dd + 63) / 64) * 4096);
      if (e == cudaSuccess) e = cudaMemset(x->attn_cnt, 0, sizeof(int) * cfg->n_heads);
      if (e == cudaSuccess) e = cudaMemset(x->gbar, 0, 64 * sizeof(unsigned));
    }
  }
  // the multi-row path (prompts of every engine, decode passes of batches): tensor maps of its GEMM operands
  if (e == cudaSuccess) {
    e = cudaFuncSetAttribute(k_gemm_tc<kTcRows>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcShape<kTcRows>::kSmemBytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_gemm_tc<kTcRowsMax>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcShape<kTcRowsMax>::kSmemBytes);
    std::vector<TensorMap128> maps;
    if (e == cudaSuccess && !build_tc_maps(x, maps)) e = cudaErrorUnknown;
    if (e == cudaSuccess) e = cudaMemcpy(x->d_tcmaps, maps.data(), sizeof(TensorMap128) * maps.size(), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_attn_rows<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_rows_smem_bytes<128>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_attn_rows<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_rows_smem_bytes<128>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_attn_rows<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_rows_smem_bytes<64>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_attn_rows<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_rows_smem_bytes<64>());
  if (e != cudaSuccess) {
    delete x;
    return ADA_ERR_CUDA;
  }
  if (cfg->ddd_threshold < 0.f && !x->use_pass) {   // the log-probabilities come from the persistent pass kernel
    delete x;
    return ADA_ERR_BAD_CONFIG;
  }
  *out = x;
  return ADA_OK;
}

extern "C" int ada_prefill(ada_ctx *x, int seq, const int32_t *d_prompt, int32_t m, int32_t *d_first_token) {
  if (!x || !d_prompt) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  if (seq < 0 || seq >= x->B) return fail(x, ADA_ERR_RANGE, "ada_prefill: seq out of range");
  if (m < 1) return fail(x, ADA_ERR_RANGE, "ada_prefill: empty prompt");
  if (m + c.n_max + 2 > c.kv_capacity) return fail(x, ADA_ERR_KV_FULL, "ada_prefill: prompt does not fit the cache");
  LAUNCH(x, k_copy_prompt, 8, 256, 0, x->tok, c.kv_capacity, seq, d_prompt, m);
  const int chunk = attn_chunk_for_prompt(m, c.kv_capacity, c.n_heads);   // attention split size of this sequence from now on
  const int last_rows = enqueue_chunks(x, seq, 0, m, m - 1, true, chunk);
  LAUNCH(x, k_finish_prefill, 1, 32, 0, x->st, x->tok, c.kv_capacity, seq, m, chunk, x->chunk_tok + (last_rows - 1),
         d_first_token);
  return finish(x, "ada_prefill");
}

extern "C" int ada_ldlp_predict(ada_ctx *x, int32_t *d_n) {
  if (!x || !d_n) return ADA_ERR_NULL;
  enqueue_ldlp(x, d_n);
  return finish(x, "ada_ldlp_predict");
}

extern "C" int ada_draft(ada_ctx *x, const int32_t *d_n, int32_t *d_draft) {
  if (!x || !d_n || !d_draft) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  if (x->has_force_n) {   // forced plain autoregressive decoding: the draft head is not kept up to date
    bool all_ar = true;
    for (int b = 0; b < x->B; ++b) all_ar = all_ar && x->host_force_n[b] == 0;
    if (all_ar) return fail(x, ADA_ERR_STATE, "ada_draft: draft lengths are forced to 0 (ada_force_n)");
  }
  LAUNCH(x, k_set_n, 1, 32, 0, x->st, d_n, x->B, c.n_max, c.kv_capacity, x->cnt);
  enqueue_draft(x);
  LAUNCH(x, k_copy_i32, 1, 128, 0, d_draft, x->draft, x->B * c.n_max);
  return finish(x, "ada_draft");
}

extern "C" int ada_label(ada_ctx *x, int32_t *d_k) {
  if (!x || !d_k) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  LAUNCH(x, k_set_n_full, 1, 32, 0, x->st, x->B, c.n_max, c.kv_capacity);
  enqueue_draft(x);
  enqueue_verify(x, -1, nullptr);
  LAUNCH(x, k_label, 1, 32, 0, x->st, x->draft, x->target, c.n_max, x->B, d_k);
  return finish(x, "ada_label");
}

extern "C" int ada_label_positions(ada_ctx *x, int seq, int32_t j0, int32_t count, int32_t *d_k, int32_t *d_drafts,
                                   int32_t *d_targets) {
  if (!x || !d_k) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  if (seq < 0 || seq >= x->B) return fail(x, ADA_ERR_RANGE, "ada_label_positions: seq out of range");
  if (j0 < 1 || count < 1) return fail(x, ADA_ERR_RANGE, "ada_label_positions: j0 >= 1 and count >= 1");
  // the sequence's lengths live on the device: this call reads them back (it synchronises the stream)
  SeqState s0;
  if (cudaMemcpyAsync(&s0, x->st + seq, sizeof(SeqState), cudaMemcpyDeviceToHost, x->stream) != cudaSuccess ||
      cudaStreamSynchronize(x->stream) != cudaSuccess)
    return fail(x, ADA_ERR_CUDA, "ada_label_positions: cannot read the sequence state");
  if (s0.len < 2) return fail(x, ADA_ERR_STATE, "ada_label_positions: the sequence has no committed tokens");
  if (j0 + count - 1 > s0.len - 1) return fail(x, ADA_ERR_RANGE, "ada_label_positions: start positions past the pending token");
  if (s0.stale || s0.len - 1 - s0.dlen > c.n_max + 1)
    return fail(x, ADA_ERR_STATE, "ada_label_positions: the draft head is behind the sequence (it was decoded without drafts)");
  // Start positions from the last to the first: the passes of position j write cache rows and features at positions
  // >= j only (draft head: >= j - 1, that row from true inputs), which no earlier start position reads.
  for (int j = j0 + count - 1; j >= j0; --j) {
    const int dl = s0.dlen < j - 1 ? s0.dlen : j - 1;
    LAUNCH(x, k_label_begin, 1, 32, 0, x->st, seq, x->B, j + 1, dl, c.n_max, c.kv_capacity);
    enqueue_draft(x);
    enqueue_verify(x, seq, nullptr);
    const int i = j - j0;
    LAUNCH(x, k_label_one, 1, 32, 0, x->st, x->draft, x->target, c.n_max, seq, d_k + i,
           d_drafts ? d_drafts + (size_t)i * c.n_max : (int *)nullptr,
           d_targets ? d_targets + (size_t)i * (c.n_max + 1) : (int *)nullptr);
  }
  // the sequence's own state again: cache rows and features from the first start position on, from the committed tokens
  LAUNCH(x, k_label_end, 1, 32, 0, x->st, seq, s0.len, s0.dlen, s0.n, s0.j_prev);
  enqueue_chunks(x, seq, j0, s0.len - 1, s0.dlen, false, s0.chunk);
  return finish(x, "ada_label_positions");
}

extern "C" int ada_draft_lengths(ada_ctx *x, int32_t *d_n) {
  if (!x || !d_n) return ADA_ERR_NULL;
  LAUNCH(x, k_gather_n, 1, 32, 0, x->st, d_n, x->B);
  return finish(x, "ada_draft_lengths");
}

extern "C" int ada_verify(ada_ctx *x, const int32_t *d_draft, const int32_t *d_n, int32_t *d_target_tok,
                          float *d_logits) {
  if (!x || !d_n || !d_target_tok) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  LAUNCH(x, k_set_n, 1, 32, 0, x->st, d_n, x->B, c.n_max, c.kv_capacity, x->cnt);
  if (d_draft && d_draft != x->draft) LAUNCH(x, k_copy_i32, 1, 128, 0, x->draft, d_draft, x->B * c.n_max);
  enqueue_verify(x, -1, d_logits);
  LAUNCH(x, k_copy_i32, 1, 128, 0, d_target_tok, x->target, x->B * (c.n_max + 1));
  return finish(x, "ada_verify");
}

extern "C" int ada_accept(ada_ctx *x, int32_t *d_accept_len, int32_t *d_emitted, int32_t *d_n_emitted) {
  if (!x) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  LAUNCH(x, k_accept, 1, 32, 0, x->st, x->tok, c.kv_capacity, x->draft, x->target, c.n_max, x->B, x->cnt, -1,
         (const int *)nullptr, 0, d_accept_len, d_emitted, d_n_emitted, (int *)nullptr);
  return finish(x, "ada_accept");
}

extern "C" int ada_step(ada_ctx *x, int32_t *d_emitted, int32_t *d_n_emitted, int32_t *d_n_used,
                        int32_t *d_accept_len) {
  if (!x) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  // the graph bakes in the override switches; re-capture when they change
  bool all_ar = x->has_force_n;  // forced plain autoregressive decoding never drafts
  for (int b = 0; b < x->B && all_ar; ++b) all_ar = x->host_force_n[b] == 0;
  const int key = (x->has_force_n ? 1 : 0) | (x->force_draft ? 2 : 0) | (all_ar ? 4 : 0);
  if (!x->graph || x->graph_key != key) {
    if (x->graph) { cudaGraphExecDestroy(x->graph); x->graph = nullptr; }
    const long long before = x->launches;
    cudaGraph_t g = nullptr;
    // record on the private stream (the caller's may be the legacy default stream, which cannot be
    // captured); the graph is then replayed on the caller's stream
    if (!x->capture_stream &&
        cudaStreamCreateWithFlags(&x->capture_stream, cudaStreamNonBlocking) != cudaSuccess)
      return fail(x, ADA_ERR_CUDA, "ada_step: cannot create the capture stream");
    cudaStream_t user_stream = x->stream;
    const int user_prof = x->prof;
    x->prof = 0;
    x->stream = x->capture_stream;
    if (cudaStreamBeginCapture(x->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      x->stream = user_stream;
      x->prof = user_prof;
      return fail(x, ADA_ERR_CUDA, "ada_step: cannot begin stream capture");
    }
    enqueue_ldlp(x, x->out_nused);
    if (!all_ar) enqueue_draft(x);
    if (!all_ar && c.ddd_threshold < 0.f)   // report the lengths the stopping rule settled on
      LAUNCH(x, k_gather_n, 1, 32, 0, x->st, x->out_nused, x->B);
    enqueue_verify(x, -1, nullptr);
    LAUNCH(x, k_accept, 1, 32, 0, x->st, x->tok, c.kv_capacity, x->draft, x->target, c.n_max, x->B, x->cnt, -1,
           (const int *)nullptr, 0, x->out_acc, x->out_emit, x->out_nemit, (int *)nullptr);
    cudaError_t e = cudaStreamEndCapture(x->stream, &g);
    x->stream = user_stream;
    x->prof = user_prof;
    x->graph_launches = (int)(x->launches - before);
    x->launches = before;
    if (e != cudaSuccess || !g) return fail(x, ADA_ERR_CUDA, "ada_step: stream capture failed");
    e = cudaGraphInstantiate(&x->graph, g, 0);
    cudaGraphDestroy(g);
    if (e != cudaSuccess) { x->graph = nullptr; return fail(x, ADA_ERR_CUDA, "ada_step: graph instantiation failed"); }
    x->graph_key = key;
  }
  if (cudaGraphLaunch(x->graph, x->stream) != cudaSuccess) return fail(x, ADA_ERR_CUDA, "ada_step: graph launch failed");
  x->launches += x->graph_launches;
  if (d_emitted) LAUNCH(x, k_copy_i32, 1, 128, 0, d_emitted, x->out_emit, x->B * (c.n_max + 1));
  if (d_n_emitted) LAUNCH(x, k_copy_i32, 1, 32, 0, d_n_emitted, x->out_nemit, x->B);
  if (d_n_used) LAUNCH(x, k_copy_i32, 1, 32, 0, d_n_used, x->out_nused, x->B);
  if (d_accept_len) LAUNCH(x, k_copy_i32, 1, 32, 0, d_accept_len, x->out_acc, x->B);
  return finish(x, "ada_step");
}

extern "C" int ada_force_n(ada_ctx *x, const int32_t *n) {
  if (!x) return ADA_ERR_NULL;
  if (!n) { x->has_force_n = 0; return ADA_OK; }
  for (int b = 0; b < x->B; ++b)
    if (n[b] < 0 || n[b] > x->c.n_max) return fail(x, ADA_ERR_RANGE, "ada_force_n: length out of range");
  for (int b = 0; b < x->B; ++b) x->host_force_n[b] = n[b];
  // pageable host memory: the copy has left the host buffer when the call returns
  if (cudaMemcpyAsync(x->force_n_dev, x->host_force_n, sizeof(int) * x->B, cudaMemcpyHostToDevice, x->stream) !=
      cudaSuccess)
    return fail(x, ADA_ERR_CUDA, "ada_force_n: copy failed");
  x->has_force_n = 1;
  return ADA_OK;
}

extern "C" int ada_force_draft(ada_ctx *x, const int32_t *d_tokens) {
  if (!x) return ADA_ERR_NULL;
  if (!d_tokens) { x->force_draft = nullptr; return ADA_OK; }
  // the tokens are copied now (stream-ordered) into a buffer of the context: the step graph keeps reading that
  // buffer, so the caller may pass a different array on every call
  if (cudaMemcpyAsync(x->forced_buf, d_tokens, sizeof(int) * x->B * x->c.n_max, cudaMemcpyDeviceToDevice, x->stream) !=
      cudaSuccess)
    return fail(x, ADA_ERR_CUDA, "ada_force_draft: copy failed");
  x->force_draft = x->forced_buf;
  return ADA_OK;
}

extern "C" int ada_force_commit(ada_ctx *x, int seq, const int32_t *d_tokens, int32_t count) {
  if (!x || !d_tokens) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  if (seq < 0 || seq >= x->B) return fail(x, ADA_ERR_RANGE, "ada_force_commit: seq out of range");
  if (count < 1 || count > c.n_max + 1) return fail(x, ADA_ERR_RANGE, "ada_force_commit: count out of range");
  LAUNCH(x, k_rewind, 1, 32, 0, x->st, seq, count, d_tokens, x->draft, c.n_max, x->cnt);
  enqueue_verify(x, seq, nullptr);
  LAUNCH(x, k_accept, 1, 32, 0, x->st, x->tok, c.kv_capacity, x->draft, x->target, c.n_max, x->B, x->cnt, seq, d_tokens,
         count, (int *)nullptr, (int *)nullptr, (int *)nullptr, (int *)nullptr);
  return finish(x, "ada_force_commit");
}

extern "C" int ada_get_counters(ada_ctx *x, int64_t out[8]) {
  if (!x || !out) return ADA_ERR_NULL;
  Counters h;
  if (cudaStreamSynchronize(x->stream) != cudaSuccess) return fail(x, ADA_ERR_CUDA, "ada_get_counters: stream error");
  if (cudaMemcpy(&h, x->cnt, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess)
    return fail(x, ADA_ERR_CUDA, "ada_get_counters: copy failed");
  out[0] = (int64_t)h.n_target; out[1] = (int64_t)h.n_draft; out[2] = (int64_t)h.n_waste; out[3] = (int64_t)h.n_tokens;
  out[4] = h.status; out[5] = x->launches; out[6] = 0; out[7] = 0;
  return ADA_OK;
}

extern "C" int ada_reset_status(ada_ctx *x) {
  if (!x) return ADA_ERR_NULL;
  if (cudaMemsetAsync(&x->cnt->status, 0, sizeof(int), x->stream) != cudaSuccess)
    return fail(x, ADA_ERR_CUDA, "ada_reset_status: memset failed");
  return ADA_OK;
}

extern "C" int ada_selftest_bounded_wait(ada_ctx *x, int32_t mode, uint32_t spin_limit, int32_t *d_result) {
  if (!x || !d_result) return ADA_ERR_NULL;
  if (mode < 0 || mode > 1 || spin_limit < 1 || spin_limit > (1u << 22))
    return fail(x, ADA_ERR_RANGE, "ada_selftest_bounded_wait: mode 0..1, 1 <= spin_limit <= 2^22");
  // a counter word of its own (not the pass kernel's), zero before the launch
  unsigned *word = x->gbar + 32;
  cudaMemsetAsync(word, 0, sizeof(unsigned), x->stream);
  LAUNCH(x, k_wait_selftest, 1, kPassThreads, 0, word, x->cnt, spin_limit, mode, d_result);
  return finish(x, "ada_selftest_bounded_wait");
}

extern "C" int ada_debug_buffer(ada_ctx *x, int which, void **d_ptr, size_t *bytes) {
  if (!x || !d_ptr || !bytes) return ADA_ERR_NULL;
  const ada_config &c = x->c;
  const size_t B = x->B;
  switch (which) {
    case 0: *d_ptr = x->feat; *bytes = B * c.kv_capacity * c.d_model * sizeof(float); break;
    case 1: *d_ptr = x->ldlp_z; *bytes = B * 16 * sizeof(float); break;
    case 2: *d_ptr = x->tok; *bytes = B * c.kv_capacity * sizeof(int); break;
    case 3: *d_ptr = x->st; *bytes = B * sizeof(SeqState); break;
    case 4: *d_ptr = x->dfeat; *bytes = B * c.n_max * c.d_model * sizeof(float); break;
    case 5: *d_ptr = x->vtop; *bytes = B * (c.n_max + 1) * sizeof(float2); break;
    case 6: *d_ptr = x->dtop; *bytes = B * c.n_max * sizeof(float2); break;
    case 7: *d_ptr = x->draft; *bytes = B * c.n_max * sizeof(int); break;
    case 8: *d_ptr = x->target; *bytes = B * (c.n_max + 1) * sizeof(int); break;
    case 10: *d_ptr = x->dlp; *bytes = B * c.n_max * sizeof(float); break;
    case 9: *d_ptr = x->phase_ns; *bytes = (512 + 4 * 512) * sizeof(unsigned long long); break;
    default: return fail(x, ADA_ERR_RANGE, "ada_debug_buffer: unknown buffer");
  }
  return ADA_OK;
}

extern "C" int ada_profile(ada_ctx *x, int enable) {
  if (!x) return ADA_ERR_NULL;
  if (enable && x->ev_pool.empty()) {
    x->ev_pool.resize(8192);
    for (auto &e : x->ev_pool)
      if (cudaEventCreate(&e) != cudaSuccess) return fail(x, ADA_ERR_CUDA, "ada_profile: cannot create events");
  }
  x->prof = enable ? 1 : 0;
  x->ev_used = 0;
  x->prof_recs.clear();
  return ADA_OK;
}

extern "C" int ada_get_profile(ada_ctx *x, double out[8]) {
  if (!x || !out) return ADA_ERR_NULL;
  if (cudaStreamSynchronize(x->stream) != cudaSuccess) return fail(x, ADA_ERR_CUDA, "ada_get_profile: stream error");
  for (int i = 0; i < 8; ++i) out[i] = 0.0;
  for (const auto &r : x->prof_recs) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, x->ev_pool[r.ev], x->ev_pool[r.ev + 1]) != cudaSuccess) continue;
    const int o = r.cls == 0 ? 0 : 3;
    out[o] += 1.0; out[o + 1] += ms; out[o + 2] += r.bytes;
  }
  return ADA_OK;
}

extern "C" const char *ada_last_error(const ada_ctx *x) { return x ? x->err.c_str() : ""; }

extern "C" int ada_destroy(ada_ctx *x) {
  if (!x) return ADA_ERR_NULL;
  cudaStreamSynchronize(x->stream);
  if (x->graph) cudaGraphExecDestroy(x->graph);
  if (x->capture_stream) cudaStreamDestroy(x->capture_stream);
  for (auto &e : x->ev_pool) cudaEventDestroy(e);
  delete x;
  return ADA_OK;
}
