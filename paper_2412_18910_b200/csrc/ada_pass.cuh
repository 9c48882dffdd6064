// Persistent whole-pass kernel for passes of at most 16 rows (batch 1): one CTA per SM runs
// every phase of a model pass (embedding or draft-head input, all decoder layers, final norm,
// LM head with greedy choice) with grid barriers between dependent phases.
//
// Why: a 7B verify pass streams 13.2 GB of weights in about 2 ms at HBM speed; one layer is ~60 us.
// Nine separate launches per layer lose a large share of that to launch gaps, ramp-up and tails.
// Here each CTA owns a fixed slab of rows of every weight matrix (N / gridDim rows), and two
// producer threads stream those slabs through a shared-memory ring with TMA tiled loads
// (cp.async.bulk.tensor.2d, 128-byte swizzle, mbarrier transaction counts; one 4 KB box per
// instruction -- separate 512-byte bulk copies were measured to cap a CTA near 12 GB/s).  Weights do not depend on activations, so the
// producer runs ahead across phase boundaries: while the other warps sit in a grid barrier or in
// the attention phase, the ring is already filling with the next GEMM's weights.
//
// Every GEMM input lives in global memory already split into two bf16 planes (hi, lo) and already in
// the swizzled tile layout the tensor core reads, written by the epilogue that produced it, so a
// whole 256-k chunk of activations is one plain 16 KB bulk copy (tiled TMA loads of 128-byte rows
// were measured to run out of request rate when activations shared them with the weights).  RMSNorm is folded around the GEMM: the producing epilogue stores split(h * gain) and
// the per-row sum of squares; the consuming epilogue multiplies its accumulators by 1/rms(row).
//
// The contraction runs on the 5th-generation tensor cores: one thread issues tcgen05.mma
// (M = 128 weight rows, N = 32 = 16 activation rows in a hi and a lo bf16 plane, K = 16) straight
// from the swizzled shared-memory tiles that TMA wrote, accumulating in tensor memory over the
// whole K range; tcgen05.commit releases ring stages and signals the finished accumulator.  (With
// mma.sync the same loop was bound by the latency of dependent register accumulators at about
// 40 % of the streaming rate.)
//
// Roles inside a CTA (12 warps):
//   warps 0, 3    weight producers, one thread each: both walk the static schedule of (phase, k chunk,
//                 k boxes, m tile) stages; warp 0 loads the even stages, warp 3 the odd ones (a single
//                 thread's mbarrier / TMA issue latency, about 700 cycles per stage, was the limit of the loops)
//   warp 1        activation producer: per GEMM phase (after the grid barrier that makes its input
//                 visible) copies the input planes chunk by chunk into shared memory
//   warp 2        one elected thread issues every tcgen05.mma and commit, in schedule order; the warp
//                 also owns the tensor-memory allocation
//   warps 4..11   workers: epilogues out of tensor memory (tcgen05.ld: one weight row per thread),
//                 attention (mma.sync on the 16-bit cache elements), row-wise phases
//
// Every wait (mbarrier, grid barrier) is bounded; when a bound is hit the kernel sets a status bit
// and carries on as if the wait had succeeded, so it always terminates.
#pragma once
#include "ada_kernels.cuh"
#include "ada_ring.h"

namespace ada {

constexpr int kPassThreads = 12 * 32;
constexpr int kNumXWarps = 1;
constexpr int kNumCWarps = 8;                    // workers
constexpr int kFirstWorker = 4;                  // warp index of worker 0
constexpr int kKc = 256;                         // k elements per activation chunk = 4 boxes of 64
constexpr int kBoxK = 64;                        // box width: 64 bf16 = 128 bytes = one swizzle row
constexpr int kStageBytes = 32 * 1024;           // largest ring stage: kb boxes of [box_rows x 64 k], kb = 2 or 4
constexpr int kXBufs = 5;
constexpr int kXBoxBytes = 32 * 128;             // activation box pair: 16 hi rows then 16 lo rows, 64 k
constexpr int kXBufBytes = (kKc / kBoxK) * kXBoxBytes;    // 16 KB per chunk
constexpr int kTmemCols = 64;                    // two accumulators of 32 columns
constexpr int kRedBytes = kNumCWarps * 32 * 8 * 4;
constexpr int kMiscBytes = 3072;                 // mbarriers and small per-CTA arrays
// attention scratch lives where the activation buffers and the reduction buffer are (both idle
// during the attention phase); the ring is NOT reused: the producer keeps filling it meanwhile
constexpr int kAttnLoopBytes = 4 * 16 * 128 * 2 + 2 * 2 * 2 * 32 * 128 * 2;   // q hi, q lo, new k, v rows; two buffers of staged keys and values
constexpr int kPassMaxSplits = 32;                // cache splits of a sequence at most (its split size is at least capacity / 32)
constexpr int kPartRow = 136;   // floats per row of a warp's partial result: 128 sums, m, l, padded so that a half-warp's fragment stores (4 rows x 4 column pairs) fall into 32 different banks
constexpr int kAttnPartBytes = 8 * 16 * kPartRow * 4 + 8 * 16 * 4 + kPassMaxSplits * 16 * 4;   // per-warp partial results, merge weights
constexpr int kAttnBytes = kAttnPartBytes > kAttnLoopBytes ? kAttnPartBytes : kAttnLoopBytes;
// (a tensor-core read of 128 tile rows may run a few KB past the last ring stage: the areas below follow the ring)
constexpr int kScratchBytes = (kXBufs * kXBufBytes + kRedBytes) > kAttnBytes ? (kXBufs * kXBufBytes + kRedBytes) : kAttnBytes;
constexpr int kPassSmemBytes = 1024 + kRingBytes + kMiscBytes + kScratchBytes;   // 1 KB to align the ring
static_assert(kPassSmemBytes <= 227 * 1024, "shared memory budget");
constexpr int kStatTimeout = 4;
constexpr unsigned kSpinLimit = 1u << 22;

struct LayerPtrs {
  const __nv_bfloat16 *wq, *wk, *wv, *wo, *wg, *wu, *wd, *na, *nm;
};

// Tensor maps (CUtensorMap, 128 bytes each) live in a device array, in this order:
//   7 per target layer (wq wk wv wo w_gate w_up w_down), 7 for the draft head's layer, then
//   eagle_fc, lm_head, then the activation planes xa_hi xa_lo at_hi at_lo ac_hi ac_lo fc_hi fc_lo.
// Weight maps: dims {K, N}, box {64, rows of one m tile of that matrix's slabs}; plane maps: dims {K, 16},
// box {64, 16}; 128-byte swizzle.
struct alignas(64) TensorMap128 {
  unsigned long long opaque[16];
};
enum { MAP_WQ = 0, MAP_WK, MAP_WV, MAP_WO, MAP_WG, MAP_WU, MAP_WD };
enum { MAPX_XA = 0, MAPX_AT = 2, MAPX_AC = 4, MAPX_FC = 6 };

struct PassParams {
  const Pass *pass;
  const TensorMap128 *maps;    // device array, see above
  int map_layer0;              // index of the first map of this pass's first layer
  int map_fc, map_lm, map_planes;
  const LayerPtrs *layers;     // device array
  int n_layers;                // layers of this pass (target: L, draft head: 1)
  int cache_layers;            // layers in the KV pool (stride)
  int d, H, hd, F, V;
  float eps;
  const __nv_bfloat16 *embed, *lm_head, *final_norm, *eagle_fc;
  int mode;                    // 0 target pass, 1 draft-head pass
  int draft_step;              // draft: 0 catch-up rows, s >= 1 single-row steps
  int with_lm;                 // run the LM head
  // activations: fp32 residual stream and qkv; bf16 (hi, lo) planes of every GEMM input
  float *h, *qkv;              // [16][d], [16][3d]
  // each input is stored as tensor-core-ready tiles (see xstore): per 64 k one 4 KB box of 32 rows
  __nv_bfloat16 *xa;              // K = d    h * gain of the norm that follows
  __nv_bfloat16 *at;              // K = d    attention output
  __nv_bfloat16 *ac;              // K = F    SwiGLU output
  __nv_bfloat16 *fc;              // K = 2d   draft-head input [e ; f]
  float *ss_part;              // [grid][16] partial sums of squares of h
  float *feat; int cap;        // target features by position [seq][cap][d]
  float *dfeat; int nmax;      // draft features [seq][nmax][d]
  // attention
  const float2 *rope;
  __nv_bfloat16 *kpool, *vpool;
  const int *page_table; int pages_per_seq, page_size;
  float *attn_part;            // [H][splits][16][hd+2]
  int *attn_cnt;               // [H] arrival counters (zero between passes)
  // LM head
  float4 *amax;                // [grid][16]
  float *logits;               // optional [slot][V]
  int *tok_out; float2 *top_out; const int *forced;
  float *lp_out;               // optional [slot]: log softmax probability of the token written to tok_out
  float *tok_logit;            // scratch [slot]: logit of a forced token (lp_out with forced tokens)
  // sync
  unsigned *gbar;              // grid barrier counter, zero at launch
  Counters *cnt;
  unsigned long long *phase_ns;  // optional [512]: [0] = start, [i+1] = time CTA 0 left barrier i (globaltimer)
};

// ---------------------------------------------------------------------------------- primitives

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait; on give-up records a status bit and returns
// (*abort_flag is a per-CTA shared word: once any wait of the CTA has given up, later waits do not spin)
// non-blocking test of the same condition (cheaper than try_wait when the phase is already complete)
__device__ __forceinline__ bool mbar_test(uint64_t *bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// (the spin is kept out of line: the kernel's phases together exceed the instruction cache, so every
// copy of cold code that is not inlined into them makes the hot part smaller)
__device__ __noinline__ void mbar_spin(uint64_t *bar, unsigned parity, Counters *cnt, volatile int *abort_flag,
                                       unsigned limit = kSpinLimit) {
  for (unsigned i = 0; i < limit; ++i) {
    if (mbar_try(bar, parity)) return;
    if (*abort_flag) return;
    if (i > 64) __nanosleep(40);
  }
  *abort_flag = 1;
  atomicOr(&cnt->status, kStatTimeout);
}
__device__ __forceinline__ void mbar_wait(uint64_t *bar, unsigned parity, Counters *cnt, volatile int *abort_flag,
                                          unsigned limit = kSpinLimit) {
  if (mbar_test(bar, parity)) return;
  mbar_spin(bar, parity, cnt, abort_flag, limit);
}
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, unsigned bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_g2s_hint(void *dst, const void *src, unsigned bytes, uint64_t *bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const TensorMap128 *map, int x, int y, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
// The same load with a level-2 eviction policy.  Weights are read once per pass: with evict-first they do not push the
// data that is read again (activation planes, partial sums, the cache) out of level 2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(void *dst, const TensorMap128 *map, int x, int y, uint64_t *bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// warp-level products on 16-bit halves with fp32 sums (attention): c[16 x 8] += a[16 x 16] b[16 x 8], and k = 8
__device__ __forceinline__ void mma_f16_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                            uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_k8(float *c, uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(b0));
}
// ---- tcgen05 (5th generation tensor cores, accumulators in tensor memory)
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_slot, uint32_t ncols) {   // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {      // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// K-major operand tile in shared memory, 128-byte swizzle: rows 128 B apart, 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// D(f32, tensor memory) (+)= A(bf16, smem) * B(bf16, smem)^T, M = 128 or 64, N = 32, K = 16
// (M = 64 for slabs of at most 64 rows: the tensor core then reads half as much of the A tile)
__host__ __device__ constexpr uint32_t umma_idesc(uint32_t m) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((32u >> 3) << 17) | ((m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// true in exactly one lane of the (converged) warp
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xffffffff;\n selp.b32 %0, 1, 0, P;\n}" : "=r"(pred));
  return pred != 0;
}
// arrive on an mbarrier once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void named_bar(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// ---- thread-block cluster of two CTAs: the peer's shared memory and its mbarriers are addressable
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t peer_addr(const void *own_smem, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(own_smem)), "r"(rank));
  return r;
}
__device__ __forceinline__ float ld_peer_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void mbar_arrive_peer(uint32_t addr) {   // releases this CTA's earlier writes to the peer
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint64_t *bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void cluster_sync_all() {   // every thread of both CTAs
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Activation tiles in global memory: for every 64 k one box of 32 rows x 128 bytes (rows 0..15 the hi
// plane of pass rows 0..15, rows 16..31 the lo plane), with the 16-byte chunk index XORed with
// (row & 7): exactly what a 128-byte-swizzle K-major operand looks like in shared memory, so a box
// (or four of them) is copied verbatim.
__device__ __forceinline__ void xstore(__nv_bfloat16 *tiles, int t, int k, float v) {
  __nv_bfloat16 hi, lo;
  split_bf16(v, hi, lo);
  const int kk = k & 63;
  const size_t o = (size_t)(k >> 6) * 2048 + (size_t)t * 64 + ((((kk >> 3) ^ (t & 7)) << 3) | (kk & 7));
  tiles[o] = hi;
  tiles[o + 16 * 64] = lo;   // row 16 + t: same (row & 7)
}

// ---------------------------------------------------------------------------------- GEMM phases

enum { EPI_STORE_QKV = 0, EPI_RESID_H = 1, EPI_SWIGLU_ACT = 2, EPI_ARGMAX_LM = 3, EPI_STORE_H = 4 };

struct GemmDesc {
  int wmap[3];                      // tensor maps of the weight matrices (segments, or gate / up)
  int nseg, Nseg, K, epi;
  const __nv_bfloat16 *xt;          // input tiles (xstore layout)
  int scale_inv_rms;                // accumulators are multiplied by 1/rms(row) of h (input was h * gain)
  int lm_rows;                      // input rows are pass->lm_row[i] (draft LM head)
  const __nv_bfloat16 *gain_next;   // RESID_H / STORE_H: planes written are split(h * gain_next); null = no gain
  int split_k;                      // this GEMM may be cut along K as well (outputs of d columns: O, down, fc)
};

// Phase list.  Target: EMBED, then per layer QKV, ATTN, O, GATEUP, DOWN, then LM.
// Draft: EAGLE_IN, FC, then the same five, then LM (optional).
enum { PH_EMBED = 0, PH_EAGLE_IN, PH_FC, PH_QKV, PH_ATTN, PH_O, PH_GATEUP, PH_DOWN, PH_LM };

__device__ __forceinline__ int phase_count(const PassParams &p) {
  return (p.mode == 0 ? 1 : 2) + 5 * p.n_layers + (p.with_lm ? 1 : 0);
}
__device__ __forceinline__ int phase_kind(const PassParams &p, int idx, int &layer) {
  layer = 0;
  const int pre = p.mode == 0 ? 1 : 2;
  if (idx < pre) return p.mode == 0 ? PH_EMBED : (idx == 0 ? PH_EAGLE_IN : PH_FC);
  const int i = idx - pre;
  if (i < 5 * p.n_layers) {
    layer = i / 5;
    return PH_QKV + (i % 5);
  }
  return PH_LM;
}

__device__ __forceinline__ bool make_gemm(const PassParams &p, int kind, int layer, GemmDesc &g) {
  const LayerPtrs &L = p.layers[layer];
  const int lm = p.map_layer0 + 7 * layer;
  g.nseg = 1; g.scale_inv_rms = 0; g.lm_rows = 0; g.gain_next = nullptr; g.split_k = 0;
  g.wmap[1] = g.wmap[2] = -1;
  switch (kind) {
    case PH_FC:
      g.wmap[0] = p.map_fc; g.Nseg = p.d; g.K = 2 * p.d; g.epi = EPI_STORE_H; g.split_k = 1;
      g.xt = p.fc; g.gain_next = L.na;
      return true;
    case PH_QKV:
      g.wmap[0] = lm + MAP_WQ; g.wmap[1] = lm + MAP_WK; g.wmap[2] = lm + MAP_WV; g.nseg = 3; g.Nseg = p.d; g.K = p.d;
      g.epi = EPI_STORE_QKV; g.xt = p.xa; g.scale_inv_rms = 1;
      return true;
    case PH_O:
      g.wmap[0] = lm + MAP_WO; g.Nseg = p.d; g.K = p.d; g.epi = EPI_RESID_H; g.split_k = 1;
      g.xt = p.at; g.gain_next = L.nm;
      return true;
    case PH_GATEUP:
      g.wmap[0] = lm + MAP_WG; g.wmap[1] = lm + MAP_WU; g.Nseg = p.F; g.K = p.d; g.epi = EPI_SWIGLU_ACT;
      g.xt = p.xa; g.scale_inv_rms = 1;
      return true;
    case PH_DOWN:
      g.wmap[0] = lm + MAP_WD; g.Nseg = p.d; g.K = p.F; g.epi = EPI_RESID_H; g.split_k = 1;
      g.xt = p.ac;
      // the norm that follows: next layer's, or the final one; the draft head has none after its layer
      g.gain_next = (layer + 1 < p.n_layers) ? p.layers[layer + 1].na : (p.mode == 0 ? p.final_norm : nullptr);
      return true;
    case PH_LM:
      g.wmap[0] = p.map_lm; g.Nseg = p.V; g.K = p.d; g.epi = EPI_ARGMAX_LM;
      g.xt = p.xa;
      if (p.mode == 0) g.scale_inv_rms = 1; else g.lm_rows = 1;
      return true;
    default:
      return false;
  }
}

// Row slab of this CTA.  A GEMM over nseg separate matrices of Nseg rows gives each matrix
// gridDim / nseg CTAs, so a slab never spans two matrices.  The slab is cut into at most two m
// tiles of box_rows <= 128 rows (the tensor map's box height, fixed per matrix at initialisation
// from the same arithmetic); SWIGLU: the two m tiles are the same row range of the gate and of the
// up matrix.  A ring stage holds kb boxes (kb * 64 k) of one m tile.
//
// GEMMs with only d output columns (O, down, the draft head's fc) would leave each CTA a slab of ~28
// rows: the tensor core then spends a whole instruction per 28 x 16 weights and every CTA re-reads the
// whole activation.  They are cut along K too: the two CTAs of a thread-block cluster share a slab of
// twice the rows, each takes one half of K (whole 256-k chunks), and the CTA of the second half adds the
// first half's partial sums, read through distributed shared memory, to its own and runs the epilogue.
struct Slab {
  int seg;          // matrix (segment) of this CTA
  int r0, rows;     // rows [r0, r0 + rows) inside that matrix
  int mtiles;       // accumulators in use (1 or 2)
  int box_rows;     // rows per m tile = box height of the tensor map
  int region;       // bytes of one box in shared memory (box_rows rounded up to 8, times 128)
  int kb;           // boxes per stage
  int m64;          // 1: M = 64 products (accumulator row i in lane (i % 16) + 32 * (i / 16))
  int ks, kj;       // K splits of this GEMM and this CTA's split
  int c0, c1;       // this CTA's 256-k chunks [c0, c1)
  int group;        // index of the slab (= group of ks CTAs)
};
__host__ __device__ __forceinline__ int slab_rpc(int Nseg, int nseg, int ncta) {
  const int cps = ncta / nseg;
  return (Nseg + cps - 1) / cps;
}
__host__ __device__ __forceinline__ int slab_box_rows(int rpc, bool swiglu) {
  const int mt = swiglu ? 1 : (rpc + 127) / 128;
  return (rpc + mt - 1) / mt;
}
// K splits for a GEMM of N output columns over K: 2 (the two CTAs of a cluster, which exchange their partial
// sums through distributed shared memory) if each split gets at least one 256-k chunk and a slab stays within
// one m tile (128 rows); else 1
__host__ __device__ __forceinline__ int slab_ksplit(int N, int K, int ncta) {
  const int nchunk = (K + kKc - 1) / kKc;
  const int groups = ncta / 2;
  if (groups < 1 || nchunk < 2) return 1;
  if ((N + groups - 1) / groups > 128) return 1;
  return 2;
}
__device__ __forceinline__ Slab make_slab(const GemmDesc &g, int cta, int ncta) {
  Slab s;
  const bool sw = g.epi == EPI_SWIGLU_ACT;
  const int nchunk = (g.K + kKc - 1) / kKc;
  s.ks = g.split_k ? slab_ksplit(g.Nseg, g.K, ncta) : 1;
  int rpc, li;
  if (s.ks > 1) {
    const int groups = ncta / s.ks;
    s.seg = 0;
    s.group = cta / s.ks;
    s.kj = cta - s.group * s.ks;
    rpc = (g.Nseg + groups - 1) / groups;
    li = s.group;
    const int per = (nchunk + s.ks - 1) / s.ks;
    s.c0 = s.kj * per;
    s.c1 = min(nchunk, s.c0 + per);
    if (s.group >= groups) { s.c0 = s.c1 = 0; li = groups; }   // CTAs beyond the last whole group idle
  } else {
    const int cps = ncta / g.nseg;                  // CTAs per matrix
    s.seg = cta / cps;
    li = cta - s.seg * cps;
    rpc = slab_rpc(g.Nseg, g.nseg, ncta);
    s.kj = 0; s.c0 = 0; s.c1 = nchunk; s.group = cta;
  }
  s.r0 = li * rpc;
  s.rows = (s.seg < g.nseg) ? max(0, min(g.Nseg, s.r0 + rpc) - s.r0) : 0;
  if (s.c1 <= s.c0) s.rows = 0;
  s.box_rows = slab_box_rows(rpc, sw);
  s.mtiles = sw ? 2 : ((rpc + 127) / 128);
  if (!sw && s.rows <= s.box_rows) s.mtiles = 1;  // a short last slab may not reach the second tile
  s.region = ((s.box_rows + 7) & ~7) * 128;
  s.kb = s.region <= 8192 ? 4 : 2;   // a stage is at most 32 KB
  s.m64 = s.box_rows <= 64;
  return s;
}
// m tile mi -> weight map index and first row
__device__ __forceinline__ void tile_source(const GemmDesc &g, const Slab &s, int mi, int &map, int &row0) {
  if (g.epi == EPI_SWIGLU_ACT) { map = g.wmap[mi]; row0 = s.r0; }
  else { map = g.wmap[s.seg]; row0 = s.r0 + mi * s.box_rows; }
}

// ---------------------------------------------------------------------------------- grid barrier

// Warp 1 and the eight worker warps (288 threads) take part; the producers' and the issuer's warps do not.
__device__ __noinline__ void grid_barrier_body(unsigned *gbar, Counters *cnt, unsigned long long *phase_ns, unsigned epoch, int tid,
                                              volatile int *abort_flag, unsigned limit = kSpinLimit) {
  named_bar(2, (kNumXWarps + kNumCWarps) * 32);
  if (tid == 32) {
    // arrive with release semantics (the named barrier above ordered the other threads' writes before this
    // thread; the release makes them visible with the count), poll with acquire loads
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(gbar) : "memory");
    const unsigned target = epoch * gridDim.x;
    bool ok = false;
    for (unsigned i = 0; i < limit && !*abort_flag; ++i) {
      if (ld_acquire(gbar) >= target) { ok = true; break; }
      if ((i & 63) == 63 && (ld_acquire(reinterpret_cast<const unsigned *>(&cnt->status)) & kStatTimeout)) break;
      if (i > 4096) __nanosleep(64);   // a barrier normally completes within a few polls
    }
    if (!ok) { *abort_flag = 1; atomicOr(&cnt->status, kStatTimeout); }
    if (phase_ns && blockIdx.x == 0 && epoch < 511) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      phase_ns[epoch] = t;
    }
  }
  named_bar(2, (kNumXWarps + kNumCWarps) * 32);
}
__device__ __forceinline__ void grid_barrier(const PassParams &p, unsigned &epoch, int tid, volatile int *abort_flag) {
  ++epoch;
  grid_barrier_body(p.gbar, p.cnt, p.phase_ns, epoch, tid, abort_flag);
}

// optional fine-grained clock of CTA 0's first consumer lane: 4 stamps per phase after the 512 barrier stamps
__device__ __forceinline__ void stamp(const PassParams &p, int ph, int k, bool on) {
  if (on && p.phase_ns && ph < 500) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    p.phase_ns[512 + 4 * ph + k] = t;
  }
}

// ---------------------------------------------------------------------------------- the kernel

__global__ void __launch_bounds__(kPassThreads, 1) k_pass(const PassParams p) {
  const int T = p.pass->T;
  if (T <= 0) return;
  const int lmT = p.pass->lmT;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;

  extern __shared__ __align__(128) unsigned char pass_smem[];
  // swizzled TMA boxes need 1024-byte aligned bases
  unsigned char *const smem = pass_smem + ((1024u - (smem_u32(pass_smem) & 1023u)) & 1023u);
  unsigned char *ring = smem;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kRingBytes);
  uint64_t *full = bars, *empty = bars + kSlots, *xfull = bars + 2 * kSlots, *xempty = bars + 2 * kSlots + kXBufs;
  float *inv_rms = reinterpret_cast<float *>(bars + 2 * kSlots + 2 * kXBufs + 4);   // [16] (after accfull and the attention barriers)
  float *ssw = inv_rms + 16;                                                       // [8][16]
  Top2 *topw = reinterpret_cast<Top2 *>(ssw + 8 * 16);                             // [8][16]
  int *flag_s = reinterpret_cast<int *>(topw + 8 * 16);
  volatile int *abort_s = flag_s + 1;
  unsigned char *xbuf = smem + kRingBytes + kMiscBytes;
  float *red = reinterpret_cast<float *>(xbuf + kXBufs * kXBufBytes);
  static_assert((2 * kSlots + 2 * kXBufs + 4) * 8 + (16 + 128) * 4 + 128 * 12 + 16 + 4 * kFlight * 4 <= kMiscBytes, "misc area");
  (void)red;

  uint64_t *accfull = xempty + kXBufs;                     // accumulator of the phase complete
  uint64_t *attn_bar = accfull + 1;                        // attention: keys and values of a round have landed (two buffers)
  uint64_t *kbar = attn_bar + 2;                           // K-split pair: the peer's partial sums are parked in its shared memory
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(const_cast<int *>(abort_s) + 1);
  uint32_t *st_rec = tmem_slot + 1;   // [2 producers][offsets, ends][kFlight]: records of the stages in flight
  if (tid == 0) {
    *abort_s = 0;
    for (int i = 0; i < kSlots; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < kXBufs; ++i) { mbar_init(&xfull[i], 1); mbar_init(&xempty[i], 1); }
    mbar_init(accfull, 1);
    mbar_init(attn_bar, 1);
    mbar_init(attn_bar + 1, 1);
    mbar_init(kbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // the two CTAs of a cluster arrive on each other's barriers later on: both must have initialised them
  cluster_sync_all();

  const int nphase = phase_count(p);
  if (p.phase_ns && cta == 0 && tid == 32) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    p.phase_ns[0] = t;
  }

  // ================================================================= weight producer
  if (warp == 0 || warp == 3) {
    if (lane != 0) return;   // one thread produces (idle lanes walking the schedule would only steal its issue slots)
    const unsigned pidx = warp == 0 ? 0u : 1u;   // producer 0 loads the even stages, producer 1 the odd ones
    uint32_t *st_off = st_rec + pidx * 2 * kFlight, *st_end = st_off + kFlight;   // this producer's own record of the stages
    RingRetire rr;   // both producers place and retire every stage of the schedule (see ada_ring.h)
    rr.init();
    const uint64_t pol_w = l2_policy_evict_first();   // weights are read once per pass
    for (int ph = 0; ph < nphase; ++ph) {
      int layer;
      const int kind = phase_kind(p, ph, layer);
      GemmDesc g;
      if (!make_gemm(p, kind, layer, g)) continue;
      if ((g.lm_rows ? lmT : T) <= 0) continue;
      const Slab s = make_slab(g, cta, ncta);
      if (s.rows == 0) continue;
      // per-phase constants in registers (tensor map and first row of each m tile)
      int map0, map1, row0, row1;
      tile_source(g, s, 0, map0, row0);
      tile_source(g, s, s.mtiles - 1, map1, row1);
      const unsigned long long m0 = reinterpret_cast<unsigned long long>(p.maps + map0);
      const unsigned long long m1 = reinterpret_cast<unsigned long long>(p.maps + map1);
      const int region = s.region, kb = s.kb, mtiles = s.mtiles, K = g.K, c1 = s.c1;
      const unsigned tx_box = (unsigned)(s.box_rows * 128);
      for (int c = s.c0; c < c1; ++c) {
        const int nbox = (min(kKc, K - c * kKc) + kBoxK - 1) / kBoxK;   // boxes that hold any k < K
        for (int b0 = 0; b0 < nbox; b0 += kb) {
          const int nb = min(kb, nbox - b0);
          for (int mi = 0; mi < mtiles; ++mi) {
            const uint32_t bytes = (uint32_t)(nb * region);
            const uint32_t off = rr.place(bytes, st_off, st_end);
            const unsigned j = rr.cur.n - 1, slot = j % kSlots;
            if ((j & 1u) != pidx) continue;   // the other producer's stage
            if (rr.pending != RingRetire::kNone) {   // stages are read in order: the newest retired one covers the rest
              mbar_wait(&empty[rr.pending % kSlots], (rr.pending / kSlots) & 1u, p.cnt, abort_s);
              rr.pending = RingRetire::kNone;
            }
            mbar_expect_tx(&full[slot], (unsigned)nb * tx_box);
            const uint32_t dst = smem_u32(ring) + off, bar = smem_u32(&full[slot]);
            const unsigned long long mp = mi ? m1 : m0;
            const int y = mi ? row1 : row0;
            for (int b = 0; b < nb; ++b)   // rows past the matrix and k past K read as zero; evict-first in level 2
              asm volatile(
                  "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(
                      dst + (uint32_t)(b * region)),
                  "l"(mp), "r"(c * kKc + (b0 + b) * kBoxK), "r"(y), "r"(bar), "l"(pol_w)
                  : "memory");
          }
        }
      }
    }
    return;
  }

  // ================================================================= tensor-core issuer (warp 2)
  // One elected thread issues every product, in schedule order (about 58 cycles per tcgen05.mma when the
  // products of a stage are issued back to back), so stages are also released in order.  M tile mi
  // accumulates in tensor-memory columns [32 mi, 32 mi + 32).
  if (warp == 2) {
    {
      RingCursor cur{0, 0};
      int xcount = 0;
      const uint32_t ring_u = smem_u32(ring), xbuf_u = smem_u32(xbuf);
      for (int ph = 0; ph < nphase; ++ph) {
        int layer;
        const int kind = phase_kind(p, ph, layer);
        GemmDesc g;
        if (!make_gemm(p, kind, layer, g)) continue;
        if ((g.lm_rows ? lmT : T) <= 0) continue;
        const Slab s = make_slab(g, cta, ncta);
        if (s.rows == 0) continue;
        const uint32_t idesc = umma_idesc(s.m64 ? 64u : 128u);
        const uint32_t region16 = (uint32_t)s.region >> 4;
        uint32_t started = 0;   // bit mi: the accumulator of m tile mi holds a product of this phase
        for (int c = s.c0; c < s.c1; ++c, ++xcount) {
          const int buf = xcount % kXBufs;
          const int kleft = min(kKc, g.K - c * kKc);
          const int nbox = (kleft + kBoxK - 1) / kBoxK;
          const uint64_t bdesc0 = umma_desc(xbuf_u + (uint32_t)buf * kXBufBytes);
          mbar_wait(&xfull[buf], (unsigned)(xcount / kXBufs) & 1u, p.cnt, abort_s);
          for (int b0 = 0; b0 < nbox; b0 += s.kb) {
            const int nb = min(s.kb, nbox - b0);
            for (int mi = 0; mi < s.mtiles; ++mi) {
              const uint32_t off = cur.take((uint32_t)(nb * s.region));
              const unsigned slot = (cur.n - 1) % kSlots, parity = ((cur.n - 1) / kSlots) & 1u;
              {
                const uint64_t adesc0 = umma_desc(ring_u + off);
                const uint32_t dcol = tmem_base + (uint32_t)mi * 32;
                mbar_wait(&full[slot], parity, p.cnt, abort_s);
                tc_fence_after();
                if (elect_one()) {   // one thread issues the stage's products and the commit that frees it
                  uint32_t acc = (started >> mi) & 1u;
                  for (int bi = 0; bi < nb; ++bi) {
                    const int box = b0 + bi;
                    const uint64_t ad = adesc0 + (uint64_t)(bi * region16);
                    const uint64_t bd = bdesc0 + (uint64_t)(box * (kXBoxBytes >> 4));
                    const int nstep = min(4, (kleft - box * kBoxK + 15) >> 4);   // k16 steps holding any k < K
                    if (nstep == 4) {
                      umma_bf16(dcol, ad, bd, idesc, acc);            // + 32 bytes per k16 step
                      umma_bf16(dcol, ad + 2, bd + 2, idesc, 1);
                      umma_bf16(dcol, ad + 4, bd + 4, idesc, 1);
                      umma_bf16(dcol, ad + 6, bd + 6, idesc, 1);
                    } else {
                      for (int s4 = 0; s4 < nstep; ++s4) umma_bf16(dcol, ad + 2 * s4, bd + 2 * s4, idesc, s4 ? 1u : acc);
                    }
                    acc = 1;
                  }
                  umma_commit(&empty[slot]);   // the stage is free once these products have read it
                }
                started |= 1u << mi;
                __syncwarp();
              }
            }
          }
          if (elect_one()) umma_commit(&xempty[buf]);
          __syncwarp();
        }
        if (elect_one()) umma_commit(accfull);
        __syncwarp();
      }
    }
    __syncwarp();
    // the workers signal when their last read of tensor memory is done
    tc_fence_before();
    named_bar(5, 32 + kNumCWarps * 32);
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
    return;
  }

  // ================================================================= activation producer + workers
  const bool is_xprod = warp == 1;
  const int cw = warp - kFirstWorker;      // worker warp index 0..7 (workers only)
  const int g8 = lane >> 2, q4 = lane & 3;
  const int ntid = is_xprod ? lane : 32 + (tid - kFirstWorker * 32);   // index among the 288 barrier participants
  const int nnth = (kNumXWarps + kNumCWarps) * 32;
  const int ctid = tid - kFirstWorker * 32;   // index among the 256 worker threads
  unsigned epoch = 0;
  int xcount = 0;   // activation chunks produced so far (buffer = xcount % kXBufs)
  unsigned acc_phase = 0;   // GEMM phases of this CTA whose accumulator has been awaited
  unsigned attn_uses[2] = {0, 0};   // completed phases of the two attention barriers
  unsigned kuses = 0;               // completed phases of the K-split pair barrier
  (void)g8; (void)q4;

  for (int ph = 0; ph < nphase; ++ph) {
    int layer;
    const int kind = phase_kind(p, ph, layer);

    // ------------------------------------------------------------- row-wise input phases
    if (kind == PH_EMBED || kind == PH_EAGLE_IN) {
      // EMBED: h = embedding rows, planes = split(h * gain of layer 0), partial sums of squares.
      // EAGLE_IN: planes of [e(token) ; feature] for the draft head's fc.  Column slices per CTA.
      const int width = kind == PH_EMBED ? p.d : 2 * p.d;
      const int cpc = (((width + ncta - 1) / ncta) + 3) & ~3;
      const int c0 = cta * cpc, c1 = min(width, c0 + cpc);
      const __nv_bfloat16 *gain = p.layers[0].na;
      for (int t = 0; t < 16; ++t) {
        float ss = 0.f;
        if (t < T) {
          const int b = p.pass->row_seq[t];
          const __nv_bfloat16 *e = p.embed + (size_t)p.pass->row_tok[t] * p.d;
          for (int c = c0 + ntid; c < c1; c += nnth) {
            if (kind == PH_EMBED) {
              const float v = __bfloat162float(e[c]);
              p.h[(size_t)t * p.d + c] = v;
              ss += v * v;
              xstore(p.xa, t, c, v * __bfloat162float(gain[c]));
            } else {
              float v;
              if (c < p.d) v = __bfloat162float(e[c]);
              else {
                const float *f = p.draft_step == 0 ? p.feat + ((size_t)b * p.cap + p.pass->row_pos[t]) * p.d
                                                   : p.dfeat + ((size_t)b * p.nmax + (p.draft_step - 1)) * p.d;
                v = __ldcg(f + (c - p.d));
              }
              xstore(p.fc, t, c, v);
            }
          }
        }
        if (kind == PH_EMBED) {
          ss = warp_sum(ss);
          if (lane == 0) red[(ntid >> 5) * 16 + t] = ss;
        }
      }
      if (kind == PH_EMBED) {
        named_bar(2, nnth);
        if (ntid < 16) {
          float sum = 0.f;
          for (int w = 0; w < kNumXWarps + kNumCWarps; ++w) sum += red[w * 16 + ntid];
          p.ss_part[(size_t)cta * 16 + ntid] = sum;
        }
      }
      grid_barrier(p, epoch, tid, abort_s);
      continue;
    }

    // ------------------------------------------------------------- attention
    if (kind == PH_ATTN) {
      if (!is_xprod) {
        // Items (head, KV split) round-robin over CTAs; one sequence on this path.  Inside an item a round
        // covers two blocks of 32 keys; warp w works on 8 keys (block w / 4, keys 8 (w % 4) .. + 8 of it) for
        // all 16 query rows with mma.sync: scores = q k^T (m16n8k16 per 16 channels), then the weighted
        // values (m16n8k8 per 8 channels).  Cache elements are 16-bit halves and enter the products as they
        // are; q and the softmax weights are fp32 and enter as a (hi, lo) pair of halves, so each product is
        // issued twice and the sums are fp32.  Keys and values of a round arrive by one bulk copy per block
        // each (a block is contiguous in its cache page) into one of two buffers, so the copies of the next
        // round fly while this one is computed.
        const int R = T, pos0 = p.pass->row_pos[0], HD = p.hd, d = p.d, half = HD >> 1;
        // The cache is cut into splits of a size fixed per sequence when its prompt was read (a multiple of 32 keys), so
        // the split a key falls in, and with it every sum of this phase, does not depend on how many rows a pass holds:
        // a row's result is the same bit for bit in a one-row pass and in a block of drafts.
        const int b = p.pass->row_seq[0];
        const int nkeys = pos0 + R, chunk = max(32, p.pass->seq_chunk[b]);
        const int nsp = min(kPassMaxSplits, (nkeys + chunk - 1) / chunk);
        __half *qh_s = reinterpret_cast<__half *>(xbuf);                              // q hi [16][128], 16-byte chunks XORed with row & 7
        __half *ql_s = qh_s + 16 * 128;                                              // q lo, same layout
        __nv_bfloat16 *k_s = reinterpret_cast<__nv_bfloat16 *>(ql_s + 16 * 128);    // new rows, rotated [16][128]
        __nv_bfloat16 *v_s = k_s + 16 * 128;
        __nv_bfloat16 *stg = v_s + 16 * 128;                                         // [2 buffers][K, V][2 blocks][32 keys][128]
        float *part_s = reinterpret_cast<float *>(xbuf);                              // [8 warps][16 rows][kPartRow], reuses the above
        float *lw_s = part_s + 8 * 16 * kPartRow;                                          // [8 warps][16 rows] merge weights
        float *wgt = lw_s + 8 * 16;                                                   // [splits][16 rows] (cross-CTA merge)
        const int g8r = lane >> 2, t4 = lane & 3;
        const int bw = cw >> 2, kq = cw & 3;
        const size_t head_stride = (size_t)kPageSize * HD;
        const uint32_t qh_u = smem_u32(qh_s), ql_u = smem_u32(ql_s);
        for (int item = cta; item < p.H * nsp; item += ncta) {
          const int hh = item / nsp, split = item - hh * nsp;
          const int kbeg = split * chunk, kend = min(nkeys, kbeg + chunk);
          const int nround = kend > kbeg ? (kend - kbeg + 63) >> 6 : 0;
          named_bar(3, kNumCWarps * 32);
          // cache pages of the item's 32-key blocks 32 i + lane, fetched 32 at a time by the first worker warp, so that
          // no copy waits for a chain of table lookups
          int pages = 0;
          if (cw == 0 && kbeg + 32 * lane < kend) pages = p.page_table[b * p.pages_per_seq + (kbeg + 32 * lane) / kPageSize];
          // round rd -> buffer rd & 1: keys then values, two blocks each (pg0, pg1: the blocks' pages)
          auto issue_round = [&](int rd, int pg0, int pg1) {
            const int r0 = kbeg + 64 * rd;
            const int nblk = min(2, (kend - r0 + 31) >> 5);
            uint64_t *bar = attn_bar + (rd & 1);
            __nv_bfloat16 *kst = stg + (size_t)(rd & 1) * 4 * 32 * 128, *vst = kst + 2 * 32 * 128;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic accesses to the buffer come first
            mbar_expect_tx(bar, (unsigned)(2 * nblk * 32 * HD * 2));
            for (int bb = 0; bb < nblk; ++bb) {
              const int key0 = r0 + 32 * bb;
              const int page = bb ? pg1 : pg0, slot = key0 % kPageSize;
              const size_t off = (((size_t)page * p.cache_layers + layer) * p.H + hh) * head_stride + (size_t)slot * HD;
              // (a layer's cache rows are read once per pass: evict-first, like the weights)
              bulk_g2s_hint(kst + (size_t)bb * 32 * HD, p.kpool + off, (unsigned)(32 * HD * 2), bar, l2_policy_evict_first());
              bulk_g2s_hint(vst + (size_t)bb * 32 * HD, p.vpool + off, (unsigned)(32 * HD * 2), bar, l2_policy_evict_first());
            }
          };
          if (cw == 0) {   // the first two rounds fly under the staging below
            const int q0 = __shfl_sync(0xffffffffu, pages, 0), q1 = __shfl_sync(0xffffffffu, pages, 1);
            const int q2 = __shfl_sync(0xffffffffu, pages, 2), q3 = __shfl_sync(0xffffffffu, pages, 3);
            if (lane == 0) {
              if (nround > 0) issue_round(0, q0, q1);
              if (nround > 1) issue_round(1, q2, q3);
            }
          }
          // q (scaled), k, v of the block rows with rotary embedding; rows past R are zero
          const float qscale = rsqrtf((float)HD);
          // (all loads of a thread's four elements, and the pages its cache rows go to, in one round trip)
          const int pos_last = pos0 + R - 1;
          int page_first = 0, page_last = 0;
          if (split == 0) {
            page_first = p.page_table[b * p.pages_per_seq + pos0 / kPageSize];
            page_last = p.page_table[b * p.pages_per_seq + pos_last / kPageSize];
          }
          for (int i0 = 0; i0 < 16 * half; i0 += 4 * kNumCWarps * 32) {
            float qa[4], qb[4], ka[4], kb[4], va[4], vb[4];
            float2 cs[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int i = i0 + u * kNumCWarps * 32 + ctid;
              const int r = i / half, c = i - r * half;
              qa[u] = qb[u] = ka[u] = kb[u] = va[u] = vb[u] = 0.f;
              cs[u] = make_float2(1.f, 0.f);
              if (i < R * half) {
                cs[u] = p.rope[(size_t)(pos0 + r) * half + c];
                const float *qr = p.qkv + (size_t)r * 3 * d + hh * HD;
                qa[u] = __ldcg(qr + c); qb[u] = __ldcg(qr + c + half);
                ka[u] = __ldcg(qr + d + c); kb[u] = __ldcg(qr + d + c + half);
                va[u] = __ldcg(qr + 2 * d + c); vb[u] = __ldcg(qr + 2 * d + c + half);
              }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int i = i0 + u * kNumCWarps * 32 + ctid;
              if (i >= 16 * half) continue;
              const int r = i / half, c = i - r * half;
              const float q0 = (qa[u] * cs[u].x - qb[u] * cs[u].y) * qscale, q1 = (qb[u] * cs[u].x + qa[u] * cs[u].y) * qscale;
              const __half h0 = __float2half_rn(q0), h1 = __float2half_rn(q1);
              const int o0 = r * 128 + ((((c >> 3) ^ (r & 7)) << 3) | (c & 7));
              const int o1 = r * 128 + (((((c + half) >> 3) ^ (r & 7)) << 3) | (c & 7));
              qh_s[o0] = h0; qh_s[o1] = h1;
              ql_s[o0] = __float2half_rn(q0 - __half2float(h0)); ql_s[o1] = __float2half_rn(q1 - __half2float(h1));
              const __nv_bfloat16 k0 = kv_store(ka[u] * cs[u].x - kb[u] * cs[u].y);   // 16-bit cache elements (see kv_store)
              const __nv_bfloat16 k1 = kv_store(kb[u] * cs[u].x + ka[u] * cs[u].y);
              const __nv_bfloat16 v0 = kv_store(va[u]), v1 = kv_store(vb[u]);
              k_s[o0] = k0; k_s[o1] = k1;      // (the staged rows have their chunks XORed by row & 7, like q)
              v_s[o0] = v0; v_s[o1] = v1;
              if (split == 0 && r < R) {  // one item per head stores the new rows in the cache
                const int pos = pos0 + r;
                // (at most 16 rows: they lie in the page of the first row or in the page of the last)
                const int page = pos / kPageSize == pos0 / kPageSize ? page_first : page_last, slot = pos % kPageSize;
                const size_t base = (((size_t)page * p.cache_layers + layer) * p.H + hh) * head_stride + (size_t)slot * HD;
                // key and value rows are stored with their 16-byte chunks XORed by (slot & 7): copied verbatim to
                // shared memory, eight consecutive rows then sit in eight different bank groups (ldmatrix of 8 keys'
                // chunk, plain for the scores and transposed for the weighted values, is conflict-free)
                const int sw = slot & 7;
                p.kpool[base + ((((c >> 3) ^ sw) << 3) | (c & 7))] = k0;
                p.kpool[base + (((((c + half) >> 3) ^ sw) << 3) | (c & 7))] = k1;
                p.vpool[base + ((((c >> 3) ^ sw) << 3) | (c & 7))] = v0;
                p.vpool[base + (((((c + half) >> 3) ^ sw) << 3) | (c & 7))] = v1;
              }
            }
          }
          // running maxima, sums and outputs of rows g8r and g8r + 8 over this warp's keys
          float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
          float o[16][4];
#pragma unroll
          for (int nt = 0; nt < 16; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
          named_bar(3, kNumCWarps * 32);   // staging visible
          for (int rd = 0; rd < nround; ++rd) {
            const int r0 = kbeg + 64 * rd;
            const int nblk = min(2, (kend - r0 + 31) >> 5);
            const __nv_bfloat16 *kst = stg + (size_t)(rd & 1) * 4 * 32 * 128, *vst = kst + 2 * 32 * 128;
            // keys and values of this round have landed (every worker keeps the barriers' parity in step)
            mbar_wait(attn_bar + (rd & 1), (attn_uses[rd & 1]++) & 1u, p.cnt, abort_s);
            const int key0 = r0 + 32 * bw + 8 * kq;     // first of this warp's 8 keys
            if (bw < nblk && key0 < kend) {
              // ---- scores: 16 rows x 8 keys
              float sc[4] = {0.f, 0.f, 0.f, 0.f}, scl[4] = {0.f, 0.f, 0.f, 0.f};   // hi and lo products apart: two chains of 8
              const int myk = key0 + (lane & 7);          // key whose row address this lane supplies
              const bool fresh = myk >= pos0;             // a row of this pass: from the staged new rows
              const uint32_t krow = fresh ? smem_u32(k_s + (size_t)min(myk - pos0, 15) * 128)
                                          : smem_u32(kst + (size_t)(bw * 32 + 8 * kq + (lane & 7)) * HD);
              const int ksw = fresh ? ((myk - pos0) & 7) : (lane & 7);     // cache rows: slot & 7 (blocks start at multiples of 32); staged rows: row & 7
              const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
              for (int kp = 0; kp < 4; ++kp) {            // pairs of 16-channel steps
                if (kp * 32 < HD) {
                  uint32_t kb0, kb1, kb2, kb3;
                  ldmatrix_x4(krow + ((((kp * 4 + (lane >> 3)) ^ ksw)) << 4), kb0, kb1, kb2, kb3);
#pragma unroll
                  for (int h2 = 0; h2 < 2; ++h2) {
                    const int ks = kp * 2 + h2;
                    const uint32_t aoff = (uint32_t)(arow * 256 + (((ks * 2 + (lane >> 4)) ^ (arow & 7)) << 4));
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(qh_u + aoff, a0, a1, a2, a3);
                    mma_f16_k16(sc, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
                    ldmatrix_x4(ql_u + aoff, a0, a1, a2, a3);
                    mma_f16_k16(scl, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
                  }
                }
              }
#pragma unroll
              for (int j = 0; j < 4; ++j) sc[j] += scl[j];
              // ---- online softmax: this thread holds keys kc, kc + 1 of rows g8r and g8r + 8
              const int kc = key0 + 2 * t4;
              const bool s00 = kc < kend && kc <= pos0 + g8r, s01 = kc + 1 < kend && kc + 1 <= pos0 + g8r;
              const bool s10 = kc < kend && kc <= pos0 + g8r + 8, s11 = kc + 1 < kend && kc + 1 <= pos0 + g8r + 8;
              float mx0 = fmaxf(s00 ? sc[0] : -INFINITY, s01 ? sc[1] : -INFINITY);
              float mx1 = fmaxf(s10 ? sc[2] : -INFINITY, s11 ? sc[3] : -INFINITY);
              mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
              mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
              const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
              float p00 = 0.f, p01 = 0.f, p10 = 0.f, p11 = 0.f, c0 = 1.f, c1 = 1.f;
              if (mn0 > -INFINITY) { p00 = s00 ? __expf(sc[0] - mn0) : 0.f; p01 = s01 ? __expf(sc[1] - mn0) : 0.f; c0 = __expf(m0 - mn0); }
              if (mn1 > -INFINITY) { p10 = s10 ? __expf(sc[2] - mn1) : 0.f; p11 = s11 ? __expf(sc[3] - mn1) : 0.f; c1 = __expf(m1 - mn1); }
              float ps0 = p00 + p01, ps1 = p10 + p11;
              ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1); ps1 += __shfl_xor_sync(0xffffffffu, ps1, 1);
              ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2); ps1 += __shfl_xor_sync(0xffffffffu, ps1, 2);
              l0 = l0 * c0 + ps0; l1 = l1 * c1 + ps1;
              m0 = mn0; m1 = mn1;
              // weights as (hi, lo) halves: A operand rows g8r, g8r + 8, k = keys 2 t4, 2 t4 + 1
              const __half2 ph0 = __floats2half2_rn(p00, p01), ph1 = __floats2half2_rn(p10, p11);
              const float2 pf0 = __half22float2(ph0), pf1 = __half22float2(ph1);
              const __half2 pl0 = __floats2half2_rn(p00 - pf0.x, p01 - pf0.y), pl1 = __floats2half2_rn(p10 - pf1.x, p11 - pf1.y);
              const uint32_t ah0 = *reinterpret_cast<const uint32_t *>(&ph0), ah1 = *reinterpret_cast<const uint32_t *>(&ph1);
              const uint32_t al0 = *reinterpret_cast<const uint32_t *>(&pl0), al1 = *reinterpret_cast<const uint32_t *>(&pl1);
              // ---- values: out[16 rows][HD] += w[16 x 8 keys] v[8 keys x HD]
              const uint32_t vrow = fresh ? smem_u32(v_s + (size_t)min(myk - pos0, 15) * 128)
                                          : smem_u32(vst + (size_t)(bw * 32 + 8 * kq + (lane & 7)) * HD);
#pragma unroll
              for (int nq = 0; nq < 4; ++nq) {            // four 8-channel tiles per load
                if (nq * 32 < HD) {
                  uint32_t v0, v1, v2, v3;
                  ldmatrix_x4_trans(vrow + (((nq * 4 + (lane >> 3)) ^ ksw) << 4), v0, v1, v2, v3);
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    float *oo = o[nq * 4 + j];
                    oo[0] *= c0; oo[1] *= c0; oo[2] *= c1; oo[3] *= c1;
                    const uint32_t vb = j == 0 ? v0 : j == 1 ? v1 : j == 2 ? v2 : v3;
                    mma_f16_k8(oo, ah0, ah1, vb);
                    mma_f16_k8(oo, al0, al1, vb);
                  }
                }
              }
            }
            named_bar(3, kNumCWarps * 32);   // every warp is done with this buffer
            if (cw == 0) {
              const int nb = 2 * (rd + 2);   // first block of the round that goes into the freed buffer
              if ((nb & 31) == 0) {
                const int k0 = kbeg + 32 * (nb + lane);
                pages = k0 < kend ? p.page_table[b * p.pages_per_seq + k0 / kPageSize] : 0;
              }
              const int pa = __shfl_sync(0xffffffffu, pages, nb & 31), pb = __shfl_sync(0xffffffffu, pages, (nb + 1) & 31);
              if (lane == 0 && rd + 2 < nround) issue_round(rd + 2, pa, pb);
            }
          }
          // per-warp partials -> shared (over the staging areas, which every warp has left), merged over
          // the eight warps in warp order, stored per (head, split)
#pragma unroll
          for (int nt = 0; nt < 16; ++nt)
            if (nt * 8 < HD) {
              *reinterpret_cast<float2 *>(part_s + (cw * 16 + g8r) * kPartRow + nt * 8 + 2 * t4) = make_float2(o[nt][0], o[nt][1]);
              *reinterpret_cast<float2 *>(part_s + (cw * 16 + g8r + 8) * kPartRow + nt * 8 + 2 * t4) = make_float2(o[nt][2], o[nt][3]);
            }
          if (t4 == 0) {
            part_s[(cw * 16 + g8r) * kPartRow + 128] = m0; part_s[(cw * 16 + g8r) * kPartRow + 129] = l0;
            part_s[(cw * 16 + g8r + 8) * kPartRow + 128] = m1; part_s[(cw * 16 + g8r + 8) * kPartRow + 129] = l1;
          }
          named_bar(3, kNumCWarps * 32);
          if (ctid < 16) {   // per row: maximum over the warps, each warp's weight, the merged sum
            const int r = ctid;
            float M = -INFINITY;
            for (int w8 = 0; w8 < kNumCWarps; ++w8) M = fmaxf(M, part_s[(w8 * 16 + r) * kPartRow + 128]);
            float lo = 0.f;
            for (int w8 = 0; w8 < kNumCWarps; ++w8) {
              const float mw = part_s[(w8 * 16 + r) * kPartRow + 128];
              const float e = mw > -INFINITY ? __expf(mw - M) : 0.f;
              lw_s[w8 * 16 + r] = e;
              lo += part_s[(w8 * 16 + r) * kPartRow + 129] * e;
            }
            if (r < R) {
              float *gp = p.attn_part + (((size_t)hh * nsp + split) * 16 + r) * (HD + 2);
              __stcg(gp + HD, M); __stcg(gp + HD + 1, lo);
            }
          }
          named_bar(3, kNumCWarps * 32);
          for (int i = ctid; i < R * HD; i += kNumCWarps * 32) {
            const int r = i / HD, c = i - r * HD;
            float oo = 0.f;
#pragma unroll
            for (int w8 = 0; w8 < kNumCWarps; ++w8) oo += part_s[(w8 * 16 + r) * kPartRow + c] * lw_s[w8 * 16 + r];
            __stcg(p.attn_part + (((size_t)hh * nsp + split) * 16 + r) * (HD + 2) + c, oo);
          }
          // the item that arrives last for this head merges the splits in split order
          __threadfence();
          named_bar(3, kNumCWarps * 32);
          if (ctid == 0) *flag_s = (atomicAdd(p.attn_cnt + hh, 1) == nsp - 1);
          named_bar(3, kNumCWarps * 32);
          if (*flag_s) {
            __threadfence();
            // weights of the splits per row first (shared), then every output element is one pass of
            // independent loads over the splits
            if (ctid < 16 && ctid < R) {
              const int r = ctid;
              const float *gp = p.attn_part + (((size_t)hh * nsp) * 16 + r) * (HD + 2);
              const size_t sst = (size_t)16 * (HD + 2);
              // (eight splits at a time, their loads in flight together; more than eight splits only in long contexts)
              float M = -INFINITY, lo = 0.f;
              if (nsp <= 8) {   // one batch of loads serves both passes
                float ms[8], ls[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  ms[u] = u < nsp ? __ldcg(gp + u * sst + HD) : -INFINITY;
                  ls[u] = u < nsp ? __ldcg(gp + u * sst + HD + 1) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) M = fmaxf(M, ms[u]);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const float e = ms[u] > -INFINITY ? __expf(ms[u] - M) : 0.f;
                  if (u < nsp) wgt[u * 16 + r] = e;
                  lo += ls[u] * e;
                }
              } else {
                for (int s0 = 0; s0 < nsp; s0 += 8) {
                  float ms[8];
#pragma unroll
                  for (int u = 0; u < 8; ++u) ms[u] = s0 + u < nsp ? __ldcg(gp + (s0 + u) * sst + HD) : -INFINITY;
#pragma unroll
                  for (int u = 0; u < 8; ++u) M = fmaxf(M, ms[u]);
                }
                for (int s0 = 0; s0 < nsp; s0 += 8) {
                  float ms[8], ls[8];
#pragma unroll
                  for (int u = 0; u < 8; ++u) {
                    ms[u] = s0 + u < nsp ? __ldcg(gp + (s0 + u) * sst + HD) : -INFINITY;
                    ls[u] = s0 + u < nsp ? __ldcg(gp + (s0 + u) * sst + HD + 1) : 0.f;
                  }
#pragma unroll
                  for (int u = 0; u < 8; ++u) {
                    const float e = ms[u] > -INFINITY ? __expf(ms[u] - M) : 0.f;
                    if (s0 + u < nsp) wgt[(s0 + u) * 16 + r] = e;
                    lo += ls[u] * e;
                  }
                }
              }
              const float inv = 1.f / lo;
              for (int s2 = 0; s2 < nsp; ++s2) wgt[s2 * 16 + r] *= inv;
            }
            named_bar(3, kNumCWarps * 32);
            const size_t sst = (size_t)16 * (HD + 2);
            if (nsp <= 8) {
              // four output elements per thread and batch: all their splits' loads are in flight together
              for (int k0 = 0; k0 < R * HD; k0 += 4 * kNumCWarps * 32) {
                float ov[4][8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const int i = k0 + k * kNumCWarps * 32 + ctid;
                  const int r = i / HD, c = i - r * HD;
                  const float *gp = p.attn_part + (((size_t)hh * nsp) * 16 + r) * (HD + 2) + c;
#pragma unroll
                  for (int u = 0; u < 8; ++u) ov[k][u] = (i < R * HD && u < nsp) ? __ldcg(gp + u * sst) : 0.f;
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const int i = k0 + k * kNumCWarps * 32 + ctid;
                  if (i >= R * HD) continue;
                  const int r = i / HD, c = i - r * HD;
                  float oo = 0.f;
#pragma unroll
                  for (int u = 0; u < 8; ++u) oo += u < nsp ? ov[k][u] * wgt[u * 16 + r] : 0.f;
                  xstore(p.at, r, hh * HD + c, oo);
                }
              }
            } else {
              for (int i = ctid; i < R * HD; i += kNumCWarps * 32) {
                const int r = i / HD, c = i - r * HD;
                const float *gp = p.attn_part + (((size_t)hh * nsp) * 16 + r) * (HD + 2) + c;
                float oo = 0.f;
                for (int s0 = 0; s0 < nsp; s0 += 8) {
                  float ov[8];
#pragma unroll
                  for (int u = 0; u < 8; ++u) ov[u] = s0 + u < nsp ? __ldcg(gp + (s0 + u) * sst) : 0.f;
#pragma unroll
                  for (int u = 0; u < 8; ++u) oo += s0 + u < nsp ? ov[u] * wgt[(s0 + u) * 16 + r] : 0.f;
                }
                xstore(p.at, r, hh * HD + c, oo);
              }
            }
            if (ctid == 0) p.attn_cnt[hh] = 0;
          }
        }
      }
      grid_barrier(p, epoch, tid, abort_s);
      continue;
    }

    // ------------------------------------------------------------- GEMM phases
    GemmDesc g;
    make_gemm(p, kind, layer, g);
    const int Tg = g.lm_rows ? lmT : T;
    if (Tg <= 0) { grid_barrier(p, epoch, tid, abort_s); continue; }
    const Slab s = make_slab(g, cta, ncta);

    if (is_xprod) {
      // ---- activation producer: the input tiles of this GEMM, one bulk copy per 256-k chunk
      if (s.rows > 0) {
        for (int c = s.c0; c < s.c1; ++c, ++xcount) {
          const int buf = xcount % kXBufs;
          if (lane == 0) {
            if (xcount >= kXBufs) mbar_wait(&xempty[buf], ((unsigned)(xcount / kXBufs) & 1u) ^ 1u, p.cnt, abort_s);
            const int nbox = (min(kKc, g.K - c * kKc) + kBoxK - 1) / kBoxK;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the buffer doubles as attention scratch
            mbar_expect_tx(&xfull[buf], (unsigned)(nbox * kXBoxBytes));
            // (every CTA reads the same input tiles: evict-last)
            bulk_g2s_hint(xbuf + (size_t)buf * kXBufBytes, g.xt + (size_t)c * (kKc / kBoxK) * (kXBoxBytes / 2),
                          (unsigned)(nbox * kXBoxBytes), &xfull[buf], l2_policy_evict_last());
          }
          __syncwarp();
        }
      }
      grid_barrier(p, epoch, tid, abort_s);
      continue;
    }

    // ---- workers: wait for the accumulator, then the epilogue straight out of tensor memory
    const bool stamper = cta == 0 && ctid == 0;
    stamp(p, ph, 0, stamper);
    // 1/rms per row of h for phases whose input was h * gain (partials summed in CTA order)
    if (g.scale_inv_rms) {
      {   // two rows per worker warp; lanes stride over the CTAs, fixed shuffle tree
        float s0 = 0.f, s1 = 0.f;
        for (int i = lane; i < ncta; i += 32) {
          s0 += __ldcg(p.ss_part + (size_t)i * 16 + 2 * cw);
          s1 += __ldcg(p.ss_part + (size_t)i * 16 + 2 * cw + 1);
        }
        s0 = warp_sum(s0); s1 = warp_sum(s1);
        if (lane == 0) {
          inv_rms[2 * cw] = rsqrtf(s0 / (float)p.d + p.eps);
          inv_rms[2 * cw + 1] = rsqrtf(s1 / (float)p.d + p.eps);
        }
      }
      named_bar(3, kNumCWarps * 32);
    }
    if (kind == PH_LM) {
      // column slice of the feature rows: target f = h / rms * gain (kept per position); draft: the
      // head's own output rows (kept per step) -- both read by later passes
      const int cpc = (p.d + ncta - 1) / ncta;
      const int c0 = cta * cpc, c1 = min(p.d, c0 + cpc);
      for (int i = ctid; i < Tg * (c1 - c0); i += kNumCWarps * 32) {
        const int t = i / (c1 - c0), c = c0 + (i - t * (c1 - c0));
        if (p.mode == 0) {
          const float v = (__ldcg(p.h + (size_t)t * p.d + c) * inv_rms[t]) * __bfloat162float(p.final_norm[c]);
          p.feat[((size_t)p.pass->row_seq[t] * p.cap + p.pass->row_pos[t]) * p.d + c] = v;
        } else {
          const int sr = p.pass->lm_row[t];
          p.dfeat[((size_t)p.pass->row_seq[sr] * p.nmax + p.draft_step) * p.d + c] = __ldcg(p.h + (size_t)sr * p.d + c);
        }
      }
    }
    stamp(p, ph, 1, stamper);
    const bool has_ss = g.epi == EPI_RESID_H || g.epi == EPI_STORE_H;
    const bool sw = g.epi == EPI_SWIGLU_ACT;
    // thread <-> weight row: quarter = warp index mod 4 (the tensor-memory lanes this warp may read),
    // m tile = worker index / 4 (SWIGLU: the first four workers read both accumulators)
    const int quarter = warp & 3, mi = sw ? 0 : (cw >> 2);
    const int rloc = s.m64 ? (lane < 16 ? quarter * 16 + lane : 1 << 20) : quarter * 32 + lane;   // row inside the m tile
    const bool active_warp = s.rows > 0 && (sw ? cw < 4 : mi < s.mtiles);
    const int rslab = mi * s.box_rows + rloc;                   // row inside the slab
    const bool valid = active_warp && rloc < s.box_rows && rslab < s.rows;
    const int vrow = s.seg * g.Nseg + s.r0 + rslab;             // output column

    // the CTA that runs the epilogue of a K-split group is the one of the last split
    const bool reducer = s.ks > 1 && s.kj == s.ks - 1;
    // old residual values, fetched while the products run
    float hold[16];
#pragma unroll
    for (int t = 0; t < 16; ++t)
      hold[t] = (valid && (s.ks == 1 || reducer) && g.epi == EPI_RESID_H && t < Tg) ? __ldcg(p.h + (size_t)t * p.d + vrow) : 0.f;
    if (s.rows > 0) {
      mbar_wait(accfull, acc_phase & 1u, p.cnt, abort_s);
      ++acc_phase;
      tc_fence_after();
    }
    stamp(p, ph, 2, stamper);
    float yy[16], uu[16];   // this thread's weight row against the 16 pass rows (hi + lo columns added)
#pragma unroll
    for (int t = 0; t < 16; ++t) { yy[t] = 0.f; uu[t] = 0.f; }
    if (active_warp) {
      float v[32], u[32];
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mi * 32);
      tmem_ld32(taddr, v);
      if (sw) {
        tmem_ld32(taddr + 32, u);
#pragma unroll
        for (int t = 0; t < 16; ++t) uu[t] = u[t] + u[16 + t];
      }
#pragma unroll
      for (int t = 0; t < 16; ++t) yy[t] = v[t] + v[16 + t];   // accumulator column = pass row
      if (g.lm_rows) {               // draft LM head: output row t is pass row lm_row[t]
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          if (t < Tg) {
            const int col = p.pass->lm_row[t];
            float sel = 0.f;
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) sel = (cc == col) ? v[cc] + v[16 + cc] : sel;
            yy[t] = sel;
          }
        }
      }
    }
    tc_fence_before();
    bool do_epi = true;
    if (s.ks > 1 && s.rows > 0) {
      // K-split pair = the two CTAs of a cluster (same slab, same thread <-> row mapping).  The CTA of the first
      // split parks its partial sums in its own shared memory and arrives on the peer's barrier; the CTA of
      // the second split waits for that, reads them through distributed shared memory, adds its own and runs
      // the epilogue: first split + second split, the same order whoever is faster.  The parked values stay
      // untouched until the next grid barrier, which the reader passes only after it has read them.
      if (!reducer) {
        float *pk = reinterpret_cast<float *>(xbuf) + ctid;
#pragma unroll
        for (int t = 0; t < 16; ++t) pk[t * 256] = yy[t];
        named_bar(3, kNumCWarps * 32);
        if (ctid == 0) mbar_arrive_peer(peer_addr(kbar, 1));
        do_epi = false;
      } else {
        bool ok = false;
        for (unsigned i = 0; i < kSpinLimit; ++i) {
          if (mbar_try_cluster(kbar, kuses & 1u)) { ok = true; break; }
          if (*abort_s) break;
          if (i > 64) __nanosleep(40);
        }
        if (!ok) { *abort_s = 1; atomicOr(&p.cnt->status, kStatTimeout); }
        ++kuses;
        const uint32_t pk = peer_addr(reinterpret_cast<float *>(xbuf) + ctid, 0);
        if (valid) {
#pragma unroll
          for (int t = 0; t < 16; ++t) yy[t] = (t < Tg ? ld_peer_f32(pk + (uint32_t)t * 1024u) : 0.f) + yy[t];
        }
      }
    }
    // The loop over the pass rows is not unrolled (the unrolled epilogues were a sixth of the kernel's code,
    // which as a whole no longer fitted the instruction cache): each thread first parks its values in a
    // column of shared memory that only it touches (the activation buffers are idle once the accumulator
    // is complete), then walks the rows.
    float *ys = reinterpret_cast<float *>(xbuf) + ctid;   // [16][256] accumulator values
    float *us = ys + 16 * 256;                            // [16][256] up-projection values (SwiGLU)
    float *hs = us + 16 * 256;                            // [16][256] old residual values
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      ys[t * 256] = yy[t];
      if (sw) us[t * 256] = uu[t];
      if (g.epi == EPI_RESID_H) hs[t * 256] = hold[t];
    }
    const bool act = valid && do_epi;
    const float gn = (act && has_ss && g.gain_next) ? __bfloat162float(g.gain_next[vrow]) : 1.f;
    const int epi = g.epi;
#pragma unroll 1
    for (int t = 0; t < Tg; ++t) {
      const float sc = g.scale_inv_rms ? inv_rms[t] : 1.f;
      const float y = ys[t * 256] * sc;
      if (epi == EPI_STORE_QKV) {
        if (act) p.qkv[(size_t)t * 3 * p.d + vrow] = y;
      } else if (has_ss) {
        float hn = 0.f;
        if (act) {
          hn = (epi == EPI_RESID_H ? hs[t * 256] : 0.f) + y;
          p.h[(size_t)t * p.d + vrow] = hn;
          xstore(p.xa, t, vrow, hn * gn);
        }
        // squares parked in the thread's column of the (now read) old-residual area; summed per pass row below
        hs[t * 256] = hn * hn;
      } else if (sw) {
        if (act) {
          const float up = us[t * 256] * sc;
          xstore(p.ac, t, vrow, (y / (1.f + __expf(-y))) * up);
        }
      } else {  // EPI_ARGMAX_LM: the warp's two largest logits of this pass row
        Top2 b;
        b.v1 = -INFINITY; b.i1 = 0x7fffffff; b.v2 = -INFINITY;
        if (act) {
          if (p.logits) {
            const int slot_out = g.lm_rows ? p.pass->lm_out[t] : p.pass->row_out[t];
            p.logits[(size_t)slot_out * p.V + vrow] = y;
          }
          b.v1 = y; b.i1 = vrow;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) b = top2_shfl_xor(b, o);
        if (lane == 0) topw[cw * 16 + t] = b;
        if (p.lp_out) {
          // for the log-probability of the chosen token: sum of exp(logit - warp maximum), and the logit of a
          // forced token where one is given
          const float e = warp_sum(act ? __expf(y - b.v1) : 0.f);
          if (lane == 0) ssw[cw * 16 + t] = e;
          if (act && p.forced) {
            const int slot_out = g.lm_rows ? p.pass->lm_out[t] : p.pass->row_out[t];
            if (p.forced[slot_out] == vrow) p.tok_logit[slot_out] = y;
          }
        }
      }
    }
    if (has_ss) {
      // sum of squares per pass row over the CTA's 256 weight-row slots: warp w takes rows 2 w and 2 w + 1, a lane eight
      // slots of each (fixed order), one warp reduction per row instead of one per row and warp inside the loop above
      named_bar(3, kNumCWarps * 32);
      const float *sq = reinterpret_cast<const float *>(xbuf) + 2 * 16 * 256;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int t = 2 * cw + k;
        float r = 0.f;
        if (t < Tg) {
#pragma unroll
          for (int j = 0; j < 8; ++j) r += sq[t * 256 + j * 32 + lane];
        }
        r = warp_sum(r);
        if (lane == 0) p.ss_part[(size_t)cta * 16 + t] = r;
      }
    } else if (epi == EPI_ARGMAX_LM) {
      if (lane >= Tg && lane < 16) {
        Top2 b;
        b.v1 = -INFINITY; b.i1 = 0x7fffffff; b.v2 = -INFINITY;
        topw[cw * 16 + lane] = b;
      }
      named_bar(3, kNumCWarps * 32);
      if (cw == 0 && lane < 16) {
        Top2 b = topw[lane];
        for (int w = 1; w < kNumCWarps; ++w) b = top2_merge(b, topw[w * 16 + lane]);
        float se = 0.f;   // sum of exp(logit - this CTA's maximum) over the CTA's vocabulary rows
        if (p.lp_out && lane < Tg)
          for (int w = 0; w < kNumCWarps; ++w) {
            const float mw = topw[w * 16 + lane].v1;
            if (mw > -INFINITY) se += ssw[w * 16 + lane] * __expf(mw - b.v1);
          }
        p.amax[(size_t)cta * 16 + lane] = make_float4(b.v1, __int_as_float(b.i1), b.v2, se);
      }
    }
    stamp(p, ph, 3, stamper);
    grid_barrier(p, epoch, tid, abort_s);

    if (g.epi == EPI_ARGMAX_LM && cta == 0) {
      // greedy choice per row: the candidates of all CTAs merged (largest value, lowest index among equals, so
      // any merge order gives the same result).  Warp w takes rows 2w and 2w + 1, 16 lanes per row, each lane
      // the CTAs congruent to it mod 16 with all its loads in flight at once.
      const int row = 2 * cw + (lane >> 4), l16 = lane & 15;
      Top2 b;
      b.v1 = -INFINITY; b.i1 = 0x7fffffff; b.v2 = -INFINITY;
      if (row < Tg) {
        float4 c4[10];
#pragma unroll
        for (int k = 0; k < 10; ++k) {
          const int i = l16 + 16 * k;
          c4[k] = i < ncta ? __ldcg(p.amax + (size_t)i * 16 + row) : make_float4(-INFINITY, __int_as_float(0x7fffffff), -INFINITY, 0.f);
        }
#pragma unroll
        for (int k = 0; k < 10; ++k) {
          Top2 x; x.v1 = c4[k].x; x.i1 = __float_as_int(c4[k].y); x.v2 = c4[k].z;
          b = top2_merge(b, x);
        }
        for (int i = l16 + 160; i < ncta; i += 16) {   // grids beyond 160 CTAs
          const float4 c = __ldcg(p.amax + (size_t)i * 16 + row);
          Top2 x; x.v1 = c.x; x.i1 = __float_as_int(c.y); x.v2 = c.z;
          b = top2_merge(b, x);
        }
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) b = top2_shfl_xor(b, o);
      float se = 0.f;   // sum over the vocabulary of exp(logit - maximum): the CTAs' sums rescaled to the global maximum
      if (p.lp_out) {
        if (row < Tg)
          for (int i = l16; i < ncta; i += 16) {
            const float4 c = __ldcg(p.amax + (size_t)i * 16 + row);
            if (c.x > -INFINITY) se += c.w * __expf(c.x - b.v1);
          }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
      }
      if (row < Tg && l16 == 0) {
        const int slot_out = g.lm_rows ? p.pass->lm_out[row] : p.pass->row_out[row];
        p.tok_out[slot_out] = p.forced ? p.forced[slot_out] : b.i1;
        if (p.top_out) p.top_out[slot_out] = make_float2(b.v1, b.v2);
        // log softmax of the token that goes out: its logit minus (maximum + log of the sum)
        if (p.lp_out) p.lp_out[slot_out] = (p.forced ? __ldcg(p.tok_logit + slot_out) - b.v1 : 0.f) - __logf(se);
      }
    }
  }
  // let warp 2 free the tensor memory once every worker has made its last read
  if (!is_xprod) {
    tc_fence_before();
    named_bar(5, 32 + kNumCWarps * 32);
  }
}

// Self-test of the bounded waits: the same wait routines as the pass kernel, on a barrier nobody arrives at (mode 0:
// an mbarrier phase that never completes; mode 1: a grid-barrier count that is never reached), with a small limit.
// Both give up, set the time-out bit of the status word and return; result[mode] receives 1 when the wait returned.
__global__ void __launch_bounds__(kPassThreads, 1) k_wait_selftest(unsigned *gbar, Counters *cnt, unsigned limit, int mode,
                                                                   int *result) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (mode == 0) {
    if (tid == 0) {
      mbar_wait(&bar, 0u, cnt, &abort_flag, limit);
      result[0] = 1;
    }
  } else if (warp == 1 || warp >= kFirstWorker) {   // the threads that take part in the pass kernel's grid barrier
    grid_barrier_body(gbar, cnt, nullptr, 2u, tid, &abort_flag, limit);   // one CTA arrives, two are awaited
    if (tid == 32) result[1] = 1;
  }
}

}  // namespace ada
