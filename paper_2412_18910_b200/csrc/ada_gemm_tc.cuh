// Multi-row GEMM on the 5th-generation tensor cores for passes of up to ROWS rows (ROWS = 88: decode passes of a
// ragged batch; ROWS = 128: prompt chunks):
//   Y[t][n] = sum_k X[t][k] * W[n][k],  t < T <= ROWS,  W bf16 [N][K] streamed once from HBM.
//
// With this many rows the activation operand is no longer small next to the weights (88 rows x {hi, lo} = 22 KB per
// 64 k against 16 KB for 128 weight rows), so a CTA takes a tall tile -- two m tiles of 128 weight rows that share
// every activation box (SwiGLU: 128 rows of the gate and the same 128 rows of the up matrix) -- and a range of K
// (grid.y splits); level-2 to shared-memory traffic then stays below 1.7 times the weight bytes.
//
//   warp 0   producer, one thread: per 64 k one stage = weight boxes (TMA tiled loads, 128-byte swizzle, box 64 k x 128
//            rows) + the hi plane box and the lo plane box of the activations (64 k x ROWS rows each, stacked so that
//            they form one K-major operand of 2 ROWS rows); 4 stages of 54 KB (ROWS = 88) or 3 of 64 KB (ROWS = 128),
//            mbarrier transaction counts
//   warp 1   one elected thread issues tcgen05.mma (M = 128, N = 2 ROWS, K = 16) per m tile and 16 k straight from the
//            TMA-written tiles; accumulators in tensor memory (m tile i in columns [256 i, 256 i + 2 ROWS));
//            tcgen05.commit frees the stage and, at the end, signals the accumulators
//   warp 2   owns the tensor-memory allocation (512 columns)
//   warps 4..11  epilogue: thread = one weight row (tensor-memory lane), tcgen05.ld eight pass rows at a time,
//            column t (hi) + column ROWS + t (lo)
//
// Every CTA leaves its sums in a scratch buffer and a reduction kernel, launched next, adds the K splits in split
// order and runs everything up to the next GEMM's input over the whole grid (k_reduce_h, k_reduce_qkv,
// k_reduce_swiglu; a last-arriving CTA per tile doing the sum alone was measured to take longer than the products:
// 16 CTAs walking 9 x 88 x 256 values each).  Only the LM head is never split: its CTAs reduce the greedy choice.  Every output element depends only on its
// own input row and on the fixed split of K.  Every wait is bounded.
#pragma once
#include "ada_pass.cuh"

namespace ada {

constexpr int kTcRows = 88;                          // rows of a decode pass of a batch at most (8 sequences x 11 rows)
constexpr int kTcRowsMax = 128;                      // rows of a prompt chunk; row scratch, partial sums and candidates are strided by it
constexpr int kTcABytes = 128 * 128;                 // one weight box: 128 rows x 64 k bf16
constexpr int kTcThreads = 12 * 32;
constexpr int kTcTmemCols = 512;
// Shapes of the two instantiations: ROWS = 88 (N = 176, four 54 KB stages) and ROWS = 128 (N = 256, the largest N of one
// product and exactly the 2 x 256 accumulator columns; three 64 KB stages).
template <int ROWS>
struct TcShape {
  static constexpr int kN = 2 * ROWS;                          // MMA N: hi rows then lo rows
  static constexpr int kBBytes = ROWS * 128;                   // one plane box
  static constexpr int kStageBytes = 2 * kTcABytes + 2 * kBBytes;
  static constexpr int kStages = ROWS <= 88 ? 4 : 3;
  static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 256;
  static_assert(kBBytes % 1024 == 0, "the lo plane must start on a swizzle-atom boundary");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
  static_assert(kN <= 256 && kN % 16 == 0, "N of one product");
};

struct GemmTcArgs {
  const TensorMap128 *wmap[3];   // box {64 k, 128 rows}; STORE: up to 3 row segments; SWIGLU: gate, up
  const TensorMap128 *xhi_map, *xlo_map;   // planes [128][ld]: box {64 k, ROWS rows}
  int epi;                    // EPI_STORE / EPI_RESID / EPI_SWIGLU (sums go to `part`) / EPI_ARGMAX
  int nseg, Nseg, K;
  int S;                      // K splits (grid.y)
  int to_part;                // the CTA leaves its sums in `part` for a reduction kernel (always, except ARGMAX)
  float *part;                // [S][128][Ntot] partial sums (S > 1; ARGMAX is never split)
  float *logits; int ldl;     // ARGMAX: optional logits [slot][ldl]
  float4 *amax;               // ARGMAX: [tiles][128] (v1, i1, v2)
  const Pass *pass;
  int use_lm_rows;            // ARGMAX in the draft: T = pass->lmT, slots = pass->lm_out
  Counters *cnts;             // status word for waits that gave up
};

// D(f32, tensor memory) (+)= A(bf16, smem) * B(bf16, smem)^T, M = m, N = n, K = 16
__host__ __device__ constexpr uint32_t umma_idesc_mn(uint32_t m, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}
// 8 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 consecutive accumulator columns of this thread's tensor-memory lane: requested here, valid after tmem_ld_wait
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

template <int ROWS>
__global__ void __launch_bounds__(kTcThreads, 1) k_gemm_tc(const GemmTcArgs a) {
  using Sh = TcShape<ROWS>;
  constexpr int kTcStages = Sh::kStages, kTcStageBytes = Sh::kStageBytes, kTcBBytes = Sh::kBBytes, kTcN = Sh::kN;
  pdl_launch_dependents();   // the next kernel may start its prologue; it waits for this grid to complete before it reads
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool sw = a.epi == EPI_SWIGLU;

  extern __shared__ __align__(128) unsigned char tc_smem[];
  unsigned char *const smem = tc_smem + ((1024u - (smem_u32(tc_smem) & 1023u)) & 1023u);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kTcStages * kTcStageBytes);
  uint64_t *full = bars, *empty = bars + kTcStages, *accfull = bars + 2 * kTcStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kTcStages + 1);
  int *flag_s = reinterpret_cast<int *>(tmem_slot + 1);
  volatile int *abort_s = flag_s + 1;

  // tile -> segment (matrix), first weight row of each m tile
  const int tiles_per_seg = sw ? (a.Nseg + 127) / 128 : (a.Nseg + 255) / 256;
  const int seg = sw ? 0 : blockIdx.x / tiles_per_seg;
  const int tile = sw ? blockIdx.x : blockIdx.x - seg * tiles_per_seg;
  const int row0 = sw ? tile * 128 : tile * 256;                    // m tile 0
  const int row1 = sw ? row0 : row0 + 128;                          // m tile 1
  const int mtiles = sw ? 2 : (row1 < a.Nseg ? 2 : 1);
  const int kboxes = (a.K + 63) >> 6;
  const int kb0 = (int)(((long long)blockIdx.y * kboxes) / a.S), kb1 = (int)(((long long)(blockIdx.y + 1) * kboxes) / a.S);

  // The producing thread initialises the barriers and fills the first stages at once: the loads fly while the
  // tensor memory is allocated and the CTA meets at the barrier below.
  const TensorMap128 *m0 = sw ? a.wmap[0] : a.wmap[seg];
  const TensorMap128 *m1 = sw ? a.wmap[1] : a.wmap[seg];
  const unsigned tx = (unsigned)(mtiles * kTcABytes + 2 * kTcBBytes);
  // level-2 policies: the weights pass through once (evict first), every CTA of a launch reads the same plane boxes (evict
  // last); what is read again soon -- planes, partial sums -- then stays in level 2 while 400 MB of weights stream by
  // (128-row layer: 131.6 -> 106.2 us for the four GEMMs)
  const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
  auto load_weights = [&](int kb, int s) {   // arms the stage's barrier for the whole stage
    unsigned char *st = smem + (size_t)s * kTcStageBytes;
    mbar_expect_tx(&full[s], tx);
    tma_load_2d_hint(st, m0, kb * 64, row0, &full[s], pol_w);     // rows past the matrix and k past K read as zero
    if (mtiles > 1) tma_load_2d_hint(st + kTcABytes, m1, kb * 64, row1, &full[s], pol_w);
  };
  auto load_planes = [&](int kb, int s) {
    unsigned char *st = smem + (size_t)s * kTcStageBytes;
    tma_load_2d_hint(st + 2 * kTcABytes, a.xhi_map, kb * 64, 0, &full[s], pol_x);
    tma_load_2d_hint(st + 2 * kTcABytes + kTcBBytes, a.xlo_map, kb * 64, 0, &full[s], pol_x);
  };
  // Weights depend on no earlier kernel: the first stages' weight boxes are requested before this grid waits for
  // the grid before it (programmatic dependent launch), the activation boxes after; the tensor memory is allocated
  // meanwhile.  The row count read before the wait is only a hint (it may be stale): it decides whether to run ahead,
  // so that a pass without rows costs next to nothing; the count read after the wait decides what is computed.
  // Nothing else of this kernel reads or writes global memory before the wait.
  const int nfirst = min(kTcStages, kb1 - kb0);
  __shared__ int ahead_s;      // one read for the whole CTA: every thread takes the same branch
  if (tid == 0) ahead_s = (a.use_lm_rows ? a.pass->lmT : a.pass->T) > 0;
  __syncthreads();
  const bool ahead = ahead_s != 0;
  int T;
  if (tid == 0) {
    *abort_s = 0;
    for (int i = 0; i < kTcStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(accfull, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (ahead)
      for (int i = 0; i < nfirst; ++i) load_weights(kb0 + i, i);
    pdl_wait();
    T = a.use_lm_rows ? a.pass->lmT : a.pass->T;
    for (int i = 0; i < nfirst && (ahead || T > 0); ++i) {
      if (!ahead) load_weights(kb0 + i, i);
      load_planes(kb0 + i, i);     // (also for a pass that turned out empty: the armed barrier must complete)
    }
  } else {
    if (warp == 2 && ahead) tmem_alloc(tmem_slot, kTcTmemCols);
    pdl_wait();
    T = a.use_lm_rows ? a.pass->lmT : a.pass->T;
    if (warp == 2 && !ahead && T > 0) tmem_alloc(tmem_slot, kTcTmemCols);
  }
  const bool idle = T <= 0;   // a pass without rows: requested stages are awaited, nothing is computed or stored
  if (idle && !ahead) return; // (uniform over the grid) nothing was requested or allocated
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------- producer
    if (lane == 0) {
      for (int kb = kb0 + nfirst, i = nfirst; kb < kb1 && !idle; ++kb, ++i) {
        const int s = i % kTcStages;
        mbar_wait(&empty[s], ((unsigned)(i / kTcStages) & 1u) ^ 1u, a.cnts, abort_s);
        load_weights(kb, s);
        load_planes(kb, s);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- tensor-core issuer
    const uint32_t idesc = umma_idesc_mn(128u, (uint32_t)kTcN);
    if (idle)
      for (int i = 0; i < nfirst; ++i) mbar_wait(&full[i], 0u, a.cnts, abort_s);   // no copy may outlive the CTA
    for (int kb = kb0, i = 0; kb < kb1 && !idle; ++kb, ++i) {
      const int s = i % kTcStages;
      mbar_wait(&full[s], (unsigned)(i / kTcStages) & 1u, a.cnts, abort_s);
      tc_fence_after();
      if (elect_one()) {
        const uint32_t st = smem_u32(smem + (size_t)s * kTcStageBytes);
        const uint64_t bd = umma_desc(st + 2 * kTcABytes);
        const int nstep = min(4, (a.K - kb * 64 + 15) >> 4);          // k16 steps holding any k < K
        for (int mi = 0; mi < mtiles; ++mi) {
          const uint64_t ad = umma_desc(st + (uint32_t)mi * kTcABytes);
          const uint32_t dcol = tmem_base + (uint32_t)mi * 256;
          for (int k4 = 0; k4 < nstep; ++k4) umma_bf16(dcol, ad + 2 * k4, bd + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
        }
        umma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (!idle && elect_one()) umma_commit(accfull);
    __syncwarp();
  }

  if (warp >= 4 && !idle) {
    // ------------------------------------------------------------- epilogue
    const int cw = warp - 4, quarter = warp & 3;
    const int ctid = tid - 128;
    const int mi = sw ? 0 : (cw >> 2);
    const bool active_warp = sw ? cw < 4 : mi < mtiles;
    const int n = (mi ? row1 : row0) + quarter * 32 + lane;         // weight row inside the segment
    const bool valid = active_warp && n < a.Nseg;
    const int Ntot = sw ? 2 * a.Nseg : a.nseg * a.Nseg;
    const int nblk = (T + 7) >> 3;
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mi * 256);

    if (kb1 > kb0) mbar_wait(accfull, 0u, a.cnts, abort_s);
    tc_fence_after();

    // pass rows 8 j .. 8 j + 7 of this thread's weight row (LM head)
    auto from_tmem = [&](int j, float (&y)[8]) {
      float hi[8], lo[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = 0.f;
      if (!active_warp || kb1 <= kb0) return;     // (warp-uniform)
      tmem_ld8(taddr + (uint32_t)(8 * j), hi);
      tmem_ld8(taddr + (uint32_t)(ROWS + 8 * j), lo);
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = hi[i] + lo[i];
    };

    if (a.to_part) {
      // 32 pass rows per round: both planes' columns are requested before the one wait, then a warp stores 128
      // contiguous bytes (32 weight rows) per pass row.  SWIGLU: warps 4..7 take the gate tile, 8..11 the up tile.
      const int pmi = cw >> 2;
      const int pn = (sw || !pmi ? row0 : row1) + quarter * 32 + lane;
      const bool pvalid = (sw || pmi < mtiles) && pn < a.Nseg;
      const int pcol = sw ? pmi * a.Nseg + pn : seg * a.Nseg + pn;
      const uint32_t paddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(pmi * 256);
      const bool have = (sw || pmi < mtiles) && kb1 > kb0;     // (warp-uniform)
      float *pp = a.part + (size_t)blockIdx.y * kTcRowsMax * Ntot + pcol;
      for (int c0 = 0; c0 < T; c0 += 32) {
        uint32_t hi[32], lo[32];
        if (have) {
          tmem_ld32_issue(paddr + (uint32_t)c0, hi);
          tmem_ld32_issue(paddr + (uint32_t)(ROWS + c0), lo);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) hi[i] = lo[i] = 0u;
        }
        if (pvalid) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c0 + i < T) __stcg(pp + (size_t)(c0 + i) * Ntot, __uint_as_float(hi[i]) + __uint_as_float(lo[i]));
        }
      }
    } else {   // LM head (never split): the warp's two largest logits of every pass row, merged per CTA
      Top2 *s_top = reinterpret_cast<Top2 *>(smem);   // [8 warps][128]: the stages are idle by now
      named_bar(3, 256);
      for (int j = 0; j < nblk; ++j) {
        float y[8];
        from_tmem(j, y);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int t = 8 * j + i;
          if (t >= T) continue;     // (uniform over the CTA)
          Top2 b;
          b.v1 = -INFINITY; b.i1 = 0x7fffffff; b.v2 = -INFINITY;
          if (valid) {
            if (a.logits) {
              const int slot = a.use_lm_rows ? a.pass->lm_out[t] : a.pass->row_out[t];
              a.logits[(size_t)slot * a.ldl + n] = y[i];
            }
            b.v1 = y[i]; b.i1 = n;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) b = top2_shfl_xor(b, o);
          if (lane == 0) s_top[cw * kTcRowsMax + t] = b;
        }
      }
      named_bar(3, 256);
      if (ctid < T) {
        Top2 b = s_top[ctid];
        for (int w = 1; w < 8; ++w) b = top2_merge(b, s_top[w * kTcRowsMax + ctid]);
        a.amax[(size_t)blockIdx.x * kTcRowsMax + ctid] = make_float4(b.v1, __int_as_float(b.i1), b.v2, 0.f);
      }
    }
  }

  // every read of tensor memory is done: free it
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 2) tmem_dealloc(tmem_base, kTcTmemCols);
}

// ---------------------------------------------------------------------------------------------
// Reduction kernels: the K splits' partial sums added in split order, then everything that follows the GEMM up to
// the next GEMM's input, so that no row-wise kernel runs between two GEMMs of a layer.
//
// RMSNorm is folded around the GEMMs: the kernel that produces the residual stream h also stores the next GEMM's input
// planes split(h * gain) and, per row, partial sums of squares of h (one per 1024-column segment, kSsSegs slots per
// row); the kernel that consumes the next GEMM's sums multiplies them by 1 / rms(row).
constexpr int kSsSegs = 8;   // segments of 1024 columns per row (d <= 8192)

__device__ __forceinline__ float inv_rms_of(const float *ss_part, int t, int d, float eps) {
  const int nseg = (d + 1023) >> 10;
  float s = 0.f;
  for (int i = 0; i < nseg; ++i) s += __ldcg(ss_part + (size_t)t * kSsSegs + i);   // fixed order
  return rsqrtf(s / (float)d + eps);
}

// h = (resid ? h : 0) + sum of the splits; planes = split(h * gain) (if gain); partial sums of squares.
// Block (segment of 1024 columns, pass row); thread = 4 columns.
struct ReduceHArgs {
  const float *part; int S, Ntot;      // [S][128][Ntot]
  float *h; int d;                      // residual stream [rows][d]
  int resid;
  const __nv_bfloat16 *gain;            // norm that follows (null: none)
  __nv_bfloat16 *xhi, *xlo; int ldx;   // planes of the next GEMM's input
  float *ss_part;                       // [rows][kSsSegs]
  const Pass *pass;
};
__global__ void __launch_bounds__(256) k_reduce_h(const ReduceHArgs a) {
  __shared__ float sh[32];
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.y, seg = blockIdx.x;
  if (t >= a.pass->T) return;
  const int col = seg * 1024 + threadIdx.x * 4;
  float ss = 0.f;
  if (col < a.d) {
    float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp = 0; sp < a.S; ++sp) {
      const float4 v = __ldcg(reinterpret_cast<const float4 *>(a.part + ((size_t)sp * kTcRowsMax + t) * a.Ntot + col));
      y.x += v.x; y.y += v.y; y.z += v.z; y.w += v.w;
    }
    float4 *hp = reinterpret_cast<float4 *>(a.h + (size_t)t * a.d + col);
    float4 hv = y;
    if (a.resid) {
      const float4 o = *hp;
      hv.x = o.x + y.x; hv.y = o.y + y.y; hv.z = o.z + y.z; hv.w = o.w + y.w;
    }
    *hp = hv;
    ss = (hv.x * hv.x + hv.y * hv.y) + (hv.z * hv.z + hv.w * hv.w);
    if (a.gain) {
      const uint2 gg = *reinterpret_cast<const uint2 *>(a.gain + col);
      const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.x), g23 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.y);
      const float x[4] = {hv.x * __bfloat162float(g01.x), hv.y * __bfloat162float(g01.y), hv.z * __bfloat162float(g23.x),
                          hv.w * __bfloat162float(g23.y)};
      __nv_bfloat16 hi[4], lo[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) split_bf16(x[i], hi[i], lo[i]);
      uint2 ph, pl;
      ph.x = (uint32_t)__bfloat16_as_ushort(hi[0]) | ((uint32_t)__bfloat16_as_ushort(hi[1]) << 16);
      ph.y = (uint32_t)__bfloat16_as_ushort(hi[2]) | ((uint32_t)__bfloat16_as_ushort(hi[3]) << 16);
      pl.x = (uint32_t)__bfloat16_as_ushort(lo[0]) | ((uint32_t)__bfloat16_as_ushort(lo[1]) << 16);
      pl.y = (uint32_t)__bfloat16_as_ushort(lo[2]) | ((uint32_t)__bfloat16_as_ushort(lo[3]) << 16);
      *reinterpret_cast<uint2 *>(a.xhi + (size_t)t * a.ldx + col) = ph;
      *reinterpret_cast<uint2 *>(a.xlo + (size_t)t * a.ldx + col) = pl;
    }
  }
  if (a.gain) {
    ss = block_sum(ss, sh);
    if (threadIdx.x == 0) a.ss_part[(size_t)t * kSsSegs + seg] = ss;
  }
}

// QKV: sums of the splits times 1 / rms(row), then rotary embedding of q and k (rotate-half pairing), q scaled by
// 1 / sqrt(hd) to qout, k and v as 16-bit cache elements into the paged pools (rows with their 16-byte chunks XORed
// by slot & 7).  Block (group of 256 (head, i) pairs, pass row); thread = one pair (i, i + hd / 2) of one head.
struct ReduceQkvArgs {
  const float *part; int S;            // [S][128][3 d]
  const float *ss_part; float eps;
  const float2 *rope; float *qout;
  __nv_bfloat16 *kpool, *vpool;
  const int *page_table; int pages_per_seq, page_size, L, layer, H, hd;
  float qscale;
  const Pass *pass;
};
__global__ void __launch_bounds__(256) k_reduce_qkv(const ReduceQkvArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = blockIdx.y;
  if (t >= a.pass->T) return;
  const int d = a.H * a.hd, half = a.hd >> 1;
  const int idx = blockIdx.x * 256 + threadIdx.x;
  if (idx >= a.H * half) return;
  const int hh = idx / half, i = idx - hh * half, o = hh * a.hd + i;
  float v[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // q_i, q_i+half, k_i, k_i+half, v_i, v_i+half
  for (int sp = 0; sp < a.S; ++sp) {
    const float *pp = a.part + ((size_t)sp * kTcRowsMax + t) * (3 * d);
    v[0] += __ldcg(pp + o); v[1] += __ldcg(pp + o + half);
    v[2] += __ldcg(pp + d + o); v[3] += __ldcg(pp + d + o + half);
    v[4] += __ldcg(pp + 2 * d + o); v[5] += __ldcg(pp + 2 * d + o + half);
  }
  const float inv = inv_rms_of(a.ss_part, t, d, a.eps);
#pragma unroll
  for (int j = 0; j < 6; ++j) v[j] *= inv;
  const int pos = a.pass->row_pos[t], b = a.pass->row_seq[t];
  const float2 cs = a.rope[(size_t)pos * half + i];
  a.qout[(size_t)t * d + o] = (v[0] * cs.x - v[1] * cs.y) * a.qscale;
  a.qout[(size_t)t * d + o + half] = (v[1] * cs.x + v[0] * cs.y) * a.qscale;
  const int page = a.page_table[b * a.pages_per_seq + pos / kPageSize], slot = pos % kPageSize;
  const size_t base = (((size_t)page * a.L + a.layer) * a.H + hh) * kPageSize * a.hd + (size_t)slot * a.hd;
  const int sw = slot & 7;
  a.kpool[base + ((((i >> 3) ^ sw) << 3) | (i & 7))] = kv_store(v[2] * cs.x - v[3] * cs.y);
  a.kpool[base + (((((i + half) >> 3) ^ sw) << 3) | (i & 7))] = kv_store(v[3] * cs.x + v[2] * cs.y);
  a.vpool[base + ((((i >> 3) ^ sw) << 3) | (i & 7))] = kv_store(v[4]);          // value rows: the same chunk order as key rows
  a.vpool[base + (((((i + half) >> 3) ^ sw) << 3) | (i & 7))] = kv_store(v[5]);
}

// SwiGLU: gate and up sums of the splits times 1 / rms(row), silu(gate) * up as hi / lo planes.
// One thread per (pass row, 4 columns), grid-stride.
struct ReduceSwigluArgs {
  const float *part; int S, F;         // [S][128][2 F]: gate columns then up columns
  const float *ss_part; float eps; int d;
  __nv_bfloat16 *ohi, *olo; int ldo;
  const Pass *pass;
};
__global__ void __launch_bounds__(256) k_reduce_swiglu(const ReduceSwigluArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  const int T = a.pass->T;
  const int c4 = a.F >> 2;
  for (int idx = blockIdx.x * 256 + threadIdx.x; idx < T * c4; idx += gridDim.x * 256) {
    const int t = idx / c4, col = (idx - t * c4) << 2;
    float4 y = make_float4(0.f, 0.f, 0.f, 0.f), u = y;
    for (int sp = 0; sp < a.S; ++sp) {
      const float *pp = a.part + ((size_t)sp * kTcRowsMax + t) * (2 * (size_t)a.F) + col;
      const float4 v = __ldcg(reinterpret_cast<const float4 *>(pp));
      const float4 w = __ldcg(reinterpret_cast<const float4 *>(pp + a.F));
      y.x += v.x; y.y += v.y; y.z += v.z; y.w += v.w;
      u.x += w.x; u.y += w.y; u.z += w.z; u.w += w.w;
    }
    const float inv = inv_rms_of(a.ss_part, t, a.d, a.eps);
    const float yy[4] = {y.x * inv, y.y * inv, y.z * inv, y.w * inv}, uu[4] = {u.x * inv, u.y * inv, u.z * inv, u.w * inv};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) split_bf16((yy[i] / (1.f + __expf(-yy[i]))) * uu[i], hi[i], lo[i]);
    uint2 ph, pl;
    ph.x = (uint32_t)__bfloat16_as_ushort(hi[0]) | ((uint32_t)__bfloat16_as_ushort(hi[1]) << 16);
    ph.y = (uint32_t)__bfloat16_as_ushort(hi[2]) | ((uint32_t)__bfloat16_as_ushort(hi[3]) << 16);
    pl.x = (uint32_t)__bfloat16_as_ushort(lo[0]) | ((uint32_t)__bfloat16_as_ushort(lo[1]) << 16);
    pl.y = (uint32_t)__bfloat16_as_ushort(lo[2]) | ((uint32_t)__bfloat16_as_ushort(lo[3]) << 16);
    *reinterpret_cast<uint2 *>(a.ohi + (size_t)t * a.ldo + col) = ph;
    *reinterpret_cast<uint2 *>(a.olo + (size_t)t * a.ldo + col) = pl;
  }
}

}  // namespace ada
