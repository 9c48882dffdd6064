// Device kernels of the adaptive speculative-decoding iteration (sm_100a).
//
// Numerics shared by all kernels: weights are bf16, KV caches 16-bit half (see kv_store); the residual
// stream, norms, softmax, every accumulator and every GEMM output are fp32.
// A GEMM input row x is carried as two bf16 rows hi = bf16(x), lo = bf16(x - hi);
// the tensor-core product W*hi + W*lo then equals W*x to ~2^-17 relative, which
// keeps logits within 2e-2 of an fp32 evaluation over 40 layers.  Every output
// element depends only on its own input row and on a fixed split of K, never on
// how many rows share the launch, so speculative and autoregressive runs of the
// library agree bit for bit.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ada {

constexpr int kMaxBatch = 8;
constexpr int kPageSize = 64;   // positions per cache page (the configuration accepts no other): divisions by it are shifts
constexpr int kMaxRows = 128;   // rows of one pass (all sequences together)
constexpr int kAttnSplits = 8;  // KV splits per (sequence, head)
constexpr int kRowGroup = 16;   // query rows of one attention CTA (one m16 tile)

// status bits (device status word)
constexpr int kStatKvFull = 1;
constexpr int kStatStale = 2;

struct SeqState {
  int len;     // committed tokens, the last one pending (its row is not in the target cache)
  int dlen;    // draft-cache rows computed from target features
  int n;       // draft length of this iteration
  int k_acc;   // accepted drafts of the last accept
  int j_prev;  // index of the pending token when the last verify started
  int n_emit;  // tokens emitted by the last accept
  int stale;   // draft head is behind by more rows than one pass holds
  int chunk;   // keys per attention split of this sequence's caches, fixed when its prompt was read (multiple of 32)
};

struct Counters {
  unsigned long long n_target, n_draft, n_waste, n_tokens;
  int status;
  int pad;
};

// Row list of the pass being computed.  Rows of one sequence are contiguous.
struct Pass {
  int T;                   // rows in this pass
  int lmT;                 // rows that go through the LM head (draft: one per active sequence)
  int row_seq[kMaxRows];
  int row_pos[kMaxRows];   // absolute position (RoPE angle, cache row)
  int row_tok[kMaxRows];   // token whose embedding enters the row
  int row_out[kMaxRows];   // output slot of the row
  int lm_row[kMaxRows];    // draft: pass row of LM row i
  int lm_out[kMaxRows];    // draft: output slot of LM row i
  int seq_row0[kMaxBatch];
  int seq_rows[kMaxBatch];
  int seq_chunk[kMaxBatch];   // keys per attention split of the sequence (SeqState::chunk)
  int4 seq_info[kMaxBatch];   // (seq_row0, seq_rows, seq_chunk, position of the first row): one load for the attention kernels
};

// Last step of every kernel that fills a row list.
__device__ __forceinline__ void pass_seal(Pass *pass, int B) {
  for (int b = 0; b < B; ++b) {
    const int r0 = pass->seq_row0[b], n = pass->seq_rows[b];
    pass->seq_info[b] = make_int4(r0, n, pass->seq_chunk[b], n > 0 ? pass->row_pos[r0] : 0);
  }
}

// KV-cache element: 16 bits per value like the weights, but IEEE half (11-bit significand) rather than bf16
// (8-bit): with bf16 keys and values the logits of a 32-layer stack were measured 0.03-0.05 away from the
// fp32 oracle (rounding of 2^-9 per layer), with half they stay inside the 2e-2 bound.  The pools are typed
// __nv_bfloat16 only as a 16-bit container; these three functions are the only ones that interpret the bits.
__device__ __forceinline__ __nv_bfloat16 kv_store(float x) {
  return __ushort_as_bfloat16(__half_as_ushort(__float2half_rn(x)));
}
__device__ __forceinline__ float kv_lo(uint32_t pair) { return __half2float(__ushort_as_half((unsigned short)(pair & 0xffffu))); }
__device__ __forceinline__ float kv_hi(uint32_t pair) { return __half2float(__ushort_as_half((unsigned short)(pair >> 16))); }

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute may start while the
// kernel before it in the stream still runs; pdl_wait returns once that kernel has completed and its writes are
// visible (at once if there is no such dependency).  Every thread of such a kernel waits before it touches memory
// another kernel writes and before it returns, so completion of a kernel implies completion of all before it.
// pdl_launch_dependents lets the kernel after this one begin its own prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// block-wide sum for blockDim.x <= 1024, result to all threads
__device__ __forceinline__ float block_sum(float v, float *sh) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += sh[i];  // fixed order
  return t;
}

// 128-bit streaming load (read once: no level-1 allocation)
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// ---------------------------------------------------------------------------------------------
// top-2 bookkeeping for the greedy choice: (v1, i1) best value / lowest index among equals, v2 second
struct Top2 {
  float v1;
  int i1;
  float v2;
};
__device__ __forceinline__ Top2 top2_merge(Top2 a, Top2 b) {
  Top2 r;
  const bool a_wins = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 <= b.i1);
  if (a_wins) {
    r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1);
  } else {
    r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(b.v2, a.v1);
  }
  return r;
}
__device__ __forceinline__ Top2 top2_shfl_xor(Top2 a, int m) {
  Top2 b;
  b.v1 = __shfl_xor_sync(0xffffffffu, a.v1, m);
  b.i1 = __shfl_xor_sync(0xffffffffu, a.i1, m);
  b.v2 = __shfl_xor_sync(0xffffffffu, a.v2, m);
  return top2_merge(a, b);
}

// ---------------------------------------------------------------------------------------------
// Epilogues of the multi-row GEMM (ada_gemm_tc.cuh).
enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_ARGMAX = 3 };

// Final greedy choice per row: merge the per-tile candidates in tile order.
// tok_out[slot] = argmax; top_out[slot] = (top1, top2).  forced (optional) overrides the token.
__global__ void k_argmax_final(const float4 *amax, int tiles, int TP, const Pass *pass, int use_lm_rows,
                               int *tok_out, float2 *top_out, const int *forced) {
  const int T = use_lm_rows ? pass->lmT : pass->T;
  const int t = blockIdx.x;
  if (t >= T) return;
  Top2 b;
  b.v1 = -INFINITY; b.i1 = 0x7fffffff; b.v2 = -INFINITY;
  for (int i0 = threadIdx.x; i0 < tiles; i0 += 4 * 32) {   // a lane's four candidates of a round in flight together
    float4 c[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      c[u] = i0 + 32 * u < tiles ? amax[(size_t)(i0 + 32 * u) * TP + t] : make_float4(-INFINITY, __int_as_float(0x7fffffff), -INFINITY, 0.f);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      Top2 x; x.v1 = c[u].x; x.i1 = __float_as_int(c[u].y); x.v2 = c[u].z;
      b = top2_merge(b, x);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) b = top2_shfl_xor(b, o);
  if (threadIdx.x == 0) {
    const int slot = use_lm_rows ? pass->lm_out[t] : pass->row_out[t];
    tok_out[slot] = forced ? forced[slot] : b.i1;
    if (top_out) top_out[slot] = make_float2(b.v1, b.v2);
  }
}

// ---------------------------------------------------------------------------------------------
// h[t][:] = embedding of row_tok[t]; planes = split(h * gain) of the first layer's norm; the row's sum of squares
// (slot 0 of the row's segments, the others zero: see the reduction kernels of the multi-row GEMM).
__global__ void k_embed(const Pass *pass, const __nv_bfloat16 *embed, float *h, int d, const __nv_bfloat16 *gain,
                        __nv_bfloat16 *xhi, __nv_bfloat16 *xlo, int ldx, float *ss_part, int ss_segs) {
  __shared__ float sh[32];
  const int t = blockIdx.x;
  if (t >= pass->T) return;
  const __nv_bfloat16 *__restrict__ e = embed + (size_t)pass->row_tok[t] * d;
  float *__restrict__ hr = h + (size_t)t * d;
  float ss = 0.f;
#pragma unroll 8
  for (int i = threadIdx.x; i < d; i += blockDim.x) {   // (loads of a row in flight together)
    const float v = __bfloat162float(e[i]);
    hr[i] = v;
    ss += v * v;
    __nv_bfloat16 hi, lo;
    split_bf16(v * __bfloat162float(gain[i]), hi, lo);
    xhi[(size_t)t * ldx + i] = hi;
    xlo[(size_t)t * ldx + i] = lo;
  }
  ss = block_sum(ss, sh);
  if (threadIdx.x < ss_segs) ss_part[(size_t)t * ss_segs + threadIdx.x] = threadIdx.x == 0 ? ss : 0.f;
}

// x = h / sqrt(mean(h^2) + eps) * gain  ->  hi/lo halves; optionally also fp32 rows to
// feat[(seq*cap + pos)][d] (the target feature f after the final norm).
__global__ void k_rmsnorm(const Pass *pass, const float *h, const __nv_bfloat16 *gain, float eps, int d,
                          __nv_bfloat16 *xhi, __nv_bfloat16 *xlo, int ldx, float *feat, int cap) {
  __shared__ float sh[32];
  const int t = blockIdx.x;
  if (t >= pass->T) return;
  // four elements per thread and step (d is a multiple of 64), the steps unrolled so that a row's loads are in
  // flight together: one element per step ran at one level-2 round trip per step
  const float4 *__restrict__ h4 = reinterpret_cast<const float4 *>(h + (size_t)t * d);
  const int d4 = d >> 2;
  float ss = 0.f;
#pragma unroll 4
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    const float4 v = h4[i];
    ss += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
  }
  ss = block_sum(ss, sh);
  const float inv = rsqrtf(ss / (float)d + eps);
  float4 *__restrict__ fr =
      feat ? reinterpret_cast<float4 *>(feat + ((size_t)pass->row_seq[t] * cap + pass->row_pos[t]) * d) : nullptr;
  const uint2 *__restrict__ g4 = reinterpret_cast<const uint2 *>(gain);
  uint2 *__restrict__ oh = reinterpret_cast<uint2 *>(xhi + (size_t)t * ldx);
  uint2 *__restrict__ ol = reinterpret_cast<uint2 *>(xlo + (size_t)t * ldx);
#pragma unroll 4
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    const float4 v = h4[i];
    const uint2 gg = g4[i];
    const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.x), g23 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.y);
    float4 x;
    x.x = (v.x * inv) * __bfloat162float(g01.x); x.y = (v.y * inv) * __bfloat162float(g01.y);
    x.z = (v.z * inv) * __bfloat162float(g23.x); x.w = (v.w * inv) * __bfloat162float(g23.y);
    __nv_bfloat16 hi[4], lo[4];
    split_bf16(x.x, hi[0], lo[0]); split_bf16(x.y, hi[1], lo[1]);
    split_bf16(x.z, hi[2], lo[2]); split_bf16(x.w, hi[3], lo[3]);
    uint2 ph, pl;
    ph.x = (uint32_t)__bfloat16_as_ushort(hi[0]) | ((uint32_t)__bfloat16_as_ushort(hi[1]) << 16);
    ph.y = (uint32_t)__bfloat16_as_ushort(hi[2]) | ((uint32_t)__bfloat16_as_ushort(hi[3]) << 16);
    pl.x = (uint32_t)__bfloat16_as_ushort(lo[0]) | ((uint32_t)__bfloat16_as_ushort(lo[1]) << 16);
    pl.y = (uint32_t)__bfloat16_as_ushort(lo[2]) | ((uint32_t)__bfloat16_as_ushort(lo[3]) << 16);
    oh[i] = ph;
    ol[i] = pl;
    if (fr) fr[i] = x;
  }
}

// hi/lo halves of selected rows of h without normalisation (draft head output -> LM head);
// also keeps the fp32 row as the head's own feature for its next step.
__global__ void k_split_lm_rows(const Pass *pass, const float *h, int d, __nv_bfloat16 *xhi,
                                __nv_bfloat16 *xlo, int ldx, float *dfeat, int nmax, int step) {
  const int i = blockIdx.x;
  if (i >= pass->lmT) return;
  const int t = pass->lm_row[i];
  const int b = pass->row_seq[t];
  const float *__restrict__ hr = h + (size_t)t * d;
  float *__restrict__ fo = dfeat + ((size_t)b * nmax + step) * d;
  __nv_bfloat16 *__restrict__ oh = xhi + (size_t)i * ldx, *__restrict__ ol = xlo + (size_t)i * ldx;
#pragma unroll 8
  for (int c = threadIdx.x; c < d; c += blockDim.x) {   // (loads of eight steps in flight together)
    const float x = hr[c];
    __nv_bfloat16 hi, lo;
    split_bf16(x, hi, lo);
    oh[c] = hi;
    ol[c] = lo;
    fo[c] = x;
  }
}

// Keys per attention split of a sequence whose prompt has m tokens, in a cache of `cap` positions, for a model of H
// heads: as many splits as keep heads x splits within the persistent kernel's 148 CTAs (four at most: 32 heads -> 4,
// 40 heads -> 3) cover the prompt and the tokens expected after it (a quarter as many again, at least 256, within the
// capacity); at least cap / 32 so that no sequence has more than 32 splits.  Chosen once per sequence, from its prompt
// alone: the split a key falls in must not depend on the shape of the pass that reads it (a one-row step and a block of
// drafts then sum in the same order).
__host__ __device__ __forceinline__ int attn_chunk_for_prompt(int m, int cap, int H) {
  const int grow = m / 4 > 256 ? m / 4 : 256;
  const int total = m + grow < cap ? m + grow : cap;
  int nsplit = H > 0 ? 148 / H : 4;
  nsplit = nsplit < 1 ? 1 : (nsplit > 4 ? 4 : nsplit);
  int chunk = ((total + nsplit - 1) / nsplit + 31) / 32 * 32;
  const int least = ((cap + 31) / 32 + 31) / 32 * 32;
  return chunk < least ? least : chunk;
}
// The multi-row attention kernel takes at most kAttnSplits splits per sequence: its split size is the sequence's, or
// cap / kAttnSplits if that is larger (again independent of the pass).
__host__ __device__ __forceinline__ int attn_rows_chunk(int seq_chunk, int cap) {
  const int least = ((cap + kAttnSplits - 1) / kAttnSplits + 31) / 32 * 32;
  const int c = seq_chunk < 32 ? 32 : seq_chunk;
  return c < least ? least : c;
}

// Merge the cache splits in split order and emit the attention output row as hi/lo halves.
template <int HD>
__global__ void k_attn_combine(const Pass *pass, const float *part, __nv_bfloat16 *xhi, __nv_bfloat16 *xlo,
                               int ldx, int cap) {
  pdl_launch_dependents();
  pdl_wait();
  const int hh = blockIdx.x, t = blockIdx.y;
  if (t >= pass->T) return;
  const int c = threadIdx.x;
  const float *base = part + (((size_t)hh * kAttnSplits) * kMaxRows + t) * (HD + 2);
  const size_t sstride = (size_t)kMaxRows * (HD + 2);
  const int4 si = pass->seq_info[pass->row_seq[t]];
  const int nkeys = si.w + si.y;
  const int chunk = attn_rows_chunk(si.z, cap);
  const int nsp = (nkeys + chunk - 1) / chunk;  // splits that held keys (at most kAttnSplits)
  float ms[kAttnSplits], ls[kAttnSplits], os[kAttnSplits];
#pragma unroll
  for (int s = 0; s < kAttnSplits; ++s) {       // all loads first: one round trip
    ms[s] = -INFINITY; ls[s] = 0.f; os[s] = 0.f;
    if (s < nsp) { ms[s] = base[s * sstride + HD]; ls[s] = base[s * sstride + HD + 1]; os[s] = base[s * sstride + c]; }
  }
  float M = -INFINITY;
#pragma unroll
  for (int s = 0; s < kAttnSplits; ++s) M = fmaxf(M, ms[s]);
  float l = 0.f, o = 0.f;
#pragma unroll
  for (int s = 0; s < kAttnSplits; ++s)
    if (s < nsp) {
      const float e = __expf(ms[s] - M);
      l += ls[s] * e;
      o += os[s] * e;
    }
  const float x = o / l;
  __nv_bfloat16 hi, lo;
  split_bf16(x, hi, lo);
  xhi[(size_t)t * ldx + hh * HD + c] = hi;
  xlo[(size_t)t * ldx + hh * HD + c] = lo;
}

// ---------------------------------------------------------------------------------------------
// Draft-head input rows: X[t] = [embedding(row_tok[t]) ; feature] as hi/lo halves (K = 2d).
// Catch-up rows (step 0) read the target feature of their position; later steps read the head's
// own previous output dfeat[seq][step-1].
__global__ void k_eagle_input(const Pass *pass, const __nv_bfloat16 *embed, const float *feat, int cap,
                              const float *dfeat, int nmax, int step, int d, __nv_bfloat16 *xhi,
                              __nv_bfloat16 *xlo, int ldx) {
  const int t = blockIdx.x;
  if (t >= pass->T) return;
  const int b = pass->row_seq[t];
  const __nv_bfloat16 *e = embed + (size_t)pass->row_tok[t] * d;
  const float *f = step == 0 ? feat + ((size_t)b * cap + pass->row_pos[t]) * d
                             : dfeat + ((size_t)b * nmax + (step - 1)) * d;
  __nv_bfloat16 *__restrict__ oh = xhi + (size_t)t * ldx, *__restrict__ ol = xlo + (size_t)t * ldx;
  const __nv_bfloat16 *__restrict__ er = e;
  const float *__restrict__ fr = f;
#pragma unroll 8
  for (int i = threadIdx.x; i < d; i += blockDim.x) {   // (loads of eight steps in flight together)
    const __nv_bfloat16 ev = er[i];
    const float fv = fr[i];
    oh[i] = ev;
    ol[i] = __float2bfloat16_rn(0.f);
    __nv_bfloat16 hi, lo;
    split_bf16(fv, hi, lo);
    oh[d + i] = hi;
    ol[d + i] = lo;
  }
}

// ---------------------------------------------------------------------------------------------
// Length predictor (Eq. 3), class-logit form.  Stage 1: hidden unit per warp:
// h[b][u] = ReLU(W1[u] . [e(tok[len-2]) ; f[len-2]] + b1[u]).  The 2d weights of a unit are streamed with 128-bit
// loads (8 bf16 per lane and step; d is a multiple of 64), all of a lane's loads of a step in flight together.
__device__ __forceinline__ float dot8_bf16(uint4 w, uint4 x) {
  const __nv_bfloat162 *wp = reinterpret_cast<const __nv_bfloat162 *>(&w), *xp = reinterpret_cast<const __nv_bfloat162 *>(&x);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 a = __bfloat1622float2(wp[i]), c = __bfloat1622float2(xp[i]);
    s += a.x * c.x + a.y * c.y;
  }
  return s;
}
__device__ __forceinline__ float dot8_bf16_f32(uint4 w, float4 x0, float4 x1) {
  const __nv_bfloat162 *wp = reinterpret_cast<const __nv_bfloat162 *>(&w);
  const float2 a = __bfloat1622float2(wp[0]), b = __bfloat1622float2(wp[1]), c = __bfloat1622float2(wp[2]), e = __bfloat1622float2(wp[3]);
  return (a.x * x0.x + a.y * x0.y) + (b.x * x0.z + b.y * x0.w) + (c.x * x1.x + c.y * x1.y) + (e.x * x1.z + e.y * x1.w);
}
__global__ void __launch_bounds__(128) k_ldlp_hidden(const SeqState *st, const int *tok, const float *feat, int cap,
                                                     const __nv_bfloat16 *embed, const __nv_bfloat16 *w1, const __nv_bfloat16 *b1,
                                                     int d, int hid, float *hbuf) {
  const int b = blockIdx.y;
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int p = st[b].len - 2;
  if (u >= hid || p < 0) return;
  const uint4 *e8 = reinterpret_cast<const uint4 *>(embed + (size_t)tok[(size_t)b * cap + p] * d);
  const float4 *f4 = reinterpret_cast<const float4 *>(feat + ((size_t)b * cap + p) * d);
  const uint4 *we = reinterpret_cast<const uint4 *>(w1 + (size_t)u * 2 * d), *wf = we + (d >> 3);
  float s = 0.f;
  const int n8 = d >> 3;   // groups of 8 elements per half of the input
#pragma unroll 8
  for (int i = lane; i < n8; i += 32) {
    const uint4 w_e = ldg_stream(we + i), w_f = ldg_stream(wf + i);
    const uint4 xe = e8[i];
    const float4 x0 = f4[2 * i], x1 = f4[2 * i + 1];
    s += dot8_bf16(w_e, xe) + dot8_bf16_f32(w_f, x0, x1);
  }
  s = warp_sum(s);
  if (lane == 0) hbuf[(size_t)b * hid + u] = fmaxf(s + __bfloat162float(b1[u]), 0.f);
}

// Scalar form (Eq. 3), one residual block: hout = hin + ReLU(W_r hin + b_r).  One warp per unit.
__global__ void k_ldlp_block(const SeqState *st, const float *hin, float *hout, const __nv_bfloat16 *wr,
                             const __nv_bfloat16 *br, int hid) {
  const int b = blockIdx.y;
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (u >= hid || st[b].len < 2) return;
  const __nv_bfloat16 *w = wr + (size_t)u * hid;
  const float *h = hin + (size_t)b * hid;
  float s = 0.f;
  for (int i = lane; i < hid; i += 32) s += __bfloat162float(w[i]) * h[i];
  s = warp_sum(s);
  if (lane == 0) hout[(size_t)b * hid + u] = h[u] + fmaxf(s + __bfloat162float(br[u]), 0.f);
}

// Stage 2: z = W2 h + b2, then n = argmax + 1 (class form, lowest index among equals) or
// n = clip(round-half-even(z_0), k_min, n_max) (scalar form, Eq. 3), then the override and the clip to the
// cache capacity.  One CTA per sequence, one warp per output (16 warps: n_max <= 15).
__global__ void __launch_bounds__(512) k_ldlp_out(SeqState *st, const float *hbuf, const __nv_bfloat16 *w2, const __nv_bfloat16 *b2,
                                                  int hid, int nmax, int mode, int kmin, int cap, const int *force_n, int has_force,
                                                  float *zbuf, int *n_out, Counters *cnt) {
  __shared__ float zs[16];
  const int b = blockIdx.x, lane = threadIdx.x & 31, c = threadIdx.x >> 5;
  const int len = st[b].len;
  if (len < 2) { if (threadIdx.x == 0) { st[b].n = 0; if (n_out) n_out[b] = 0; } return; }
  const int nz = mode == 0 ? nmax : 1;
  if (c < nz) {
    float s = 0.f;
    for (int i = lane; i < hid; i += 32) s += __bfloat162float(w2[(size_t)c * hid + i]) * hbuf[(size_t)b * hid + i];
    s = warp_sum(s) + __bfloat162float(b2[c]);
    if (lane == 0) { zs[c] = s; zbuf[b * 16 + c] = s; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float best = -INFINITY;
    int bi = 0;
    for (int i = 0; i < nz; ++i)
      if (zs[i] > best) { best = zs[i]; bi = i; }
    int n = bi + 1;
    if (mode != 0) n = (int)fminf(fmaxf(rintf(best), (float)kmin), (float)nmax);   // best = z_0
    if (has_force) n = force_n[b];
    const int room = cap - len - 1;  // the n + 1 tokens this iteration may commit must fit: len + n + 1 <= cap
    if (n > room) { n = room < 0 ? 0 : room; atomicOr(&cnt->status, kStatKvFull); }
    st[b].n = n;
    if (n_out) n_out[b] = n;
  }
}

// n[b] <- user array (separate-call API), with the same clip
__global__ void k_set_n(SeqState *st, const int *n_in, int B, int nmax, int cap, Counters *cnt) {
  const int b = threadIdx.x;
  if (b >= B) return;
  int n = n_in[b];
  n = max(0, min(n, nmax));
  const int room = cap - st[b].len - 1;
  if (n > room) { n = room < 0 ? 0 : room; atomicOr(&cnt->status, kStatKvFull); }
  st[b].n = n;
}

// ---------------------------------------------------------------------------------------------
// Row lists.  One thread block of one warp; B <= 8, rows <= kMaxRows.
//
// Verify (Eq. 1): rows of sequence b = pending token then its n drafts, positions j..j+n.
__global__ void k_rows_verify(Pass *pass, SeqState *st, const int *tok, int cap, const int *draft, int nmax, int B,
                              int only_seq) {
  if (threadIdx.x != 0) return;
  int T = 0;
  for (int b = 0; b < B; ++b) {
    pass->seq_row0[b] = T;
    pass->seq_rows[b] = 0;
    pass->seq_chunk[b] = st[b].chunk;
    if (only_seq >= 0 && b != only_seq) continue;
    const int len = st[b].len;
    if (len < 1) continue;
    const int j = len - 1, n = st[b].n;
    if (len + n + 1 > cap) continue;  // a full sequence takes no further step
    st[b].j_prev = j;
    for (int i = 0; i <= n; ++i) {
      pass->row_seq[T] = b;
      pass->row_pos[T] = j + i;
      pass->row_tok[T] = i == 0 ? tok[(size_t)b * cap + j] : draft[b * nmax + i - 1];
      pass->row_out[T] = b * (nmax + 1) + i;
      ++T;
    }
    pass->seq_rows[b] = n + 1;
  }
  pass->T = T;
  pass->lmT = T;
  pass_seal(pass, B);
}

// Prefill chunk: rows pos0..pos0+R-1 of sequence b, tokens from the committed-token array.
__global__ void k_rows_chunk(Pass *pass, const int *tok, int cap, int b, int pos0, int R, int tok_shift, int B, int chunk) {
  if (threadIdx.x != 0) return;
  for (int i = 0; i < B; ++i) { pass->seq_row0[i] = 0; pass->seq_rows[i] = 0; pass->seq_chunk[i] = chunk; }
  for (int i = 0; i < R; ++i) {
    pass->row_seq[i] = b;
    pass->row_pos[i] = pos0 + i;
    pass->row_tok[i] = tok[(size_t)b * cap + pos0 + i + tok_shift];
    pass->row_out[i] = i;
    pass->lm_row[i] = i;
    pass->lm_out[i] = i;
  }
  pass->seq_rows[b] = R;
  pass->T = R;
  pass->lmT = R;
  pass_seal(pass, B);
}

// Draft (Eq. 2).  step 0: catch-up rows p = dlen..j-1 of every sequence with n >= 1; row p pairs the
// target feature of p with the embedding of token p+1; the last row feeds the LM head.
// step s >= 1: one row per sequence with n > s at position j+s-1, token = draft[s-1].
__global__ void k_rows_draft(Pass *pass, SeqState *st, const int *tok, int cap, const int *draft, int nmax, int B,
                             int step, int max_rows, Counters *cnt) {
  if (threadIdx.x != 0) return;
  int T = 0, lmT = 0;
  for (int b = 0; b < B; ++b) {
    pass->seq_row0[b] = T;
    pass->seq_rows[b] = 0;
    pass->seq_chunk[b] = st[b].chunk;
    const int n = st[b].n, j = st[b].len - 1;
    if (n <= step || j < 1) continue;
    if (step == 0) {
      int R = j - st[b].dlen, p0 = st[b].dlen;
      // already up to date (a second draft from the same state, e.g. after a label pass): the row of position
      // j - 1 is computed again -- same inputs, same cache row -- because its output yields the first draft token
      if (R == 0) { R = 1; p0 = j - 1; }
      if (R < 1 || T + R > max_rows || st[b].stale) { st[b].n = 0; atomicOr(&cnt->status, kStatStale); continue; }
      for (int i = 0; i < R; ++i) {
        const int p = p0 + i;
        pass->row_seq[T] = b;
        pass->row_pos[T] = p;
        pass->row_tok[T] = tok[(size_t)b * cap + p + 1];
        pass->row_out[T] = 0;
        ++T;
      }
      pass->seq_rows[b] = R;
      st[b].dlen = j;
    } else {
      pass->row_seq[T] = b;
      pass->row_pos[T] = j + step - 1;
      pass->row_tok[T] = draft[b * nmax + step - 1];
      pass->row_out[T] = 0;
      ++T;
      pass->seq_rows[b] = 1;
    }
    pass->lm_row[lmT] = T - 1;
    pass->lm_out[lmT] = b * nmax + step;
    ++lmT;
  }
  pass->T = T;
  pass->lmT = lmT;
  pass_seal(pass, B);
}

// ---------------------------------------------------------------------------------------------
// Accept (Eq. 1 and the footnote of Section 3.1) and roll-back.  One thread per sequence.
// forced_count > 0 (force_commit of sequence only_seq): accept count-1 drafts and take the bonus
// from forced_tok instead of the target's choice.
__global__ void k_accept(SeqState *st, int *tok, int cap, const int *draft, const int *target, int nmax, int B,
                         Counters *cnt, int only_seq, const int *forced_tok, int forced_count, int *acc_out,
                         int *emit_out, int *nemit_out, int *nused_out) {
  const int b = threadIdx.x;
  if (b >= B) return;
  if (only_seq >= 0 && b != only_seq) return;
  const int len = st[b].len;
  if (len < 1) return;
  const int n = st[b].n;
  const int j = st[b].j_prev;
  if (j != len - 1 || len + n + 1 > cap) {  // no verify ran for this sequence
    if (acc_out) acc_out[b] = 0;
    if (nemit_out) nemit_out[b] = 0;
    if (nused_out) nused_out[b] = n;
    st[b].n_emit = 0;
    return;
  }
  int k = 0;
  if (forced_count > 0) {
    k = forced_count - 1;
  } else {
    while (k < n && draft[b * nmax + k] == target[b * (nmax + 1) + k]) ++k;
  }
  for (int i = 0; i <= k; ++i) {
    int t;
    if (forced_count > 0) t = forced_tok[i];
    else t = i < k ? draft[b * nmax + i] : target[b * (nmax + 1) + k];
    tok[(size_t)b * cap + j + 1 + i] = t;
    if (emit_out) emit_out[b * (nmax + 1) + i] = t;
  }
  st[b].len = j + k + 2;
  st[b].k_acc = k;
  st[b].n_emit = k + 1;
  if (n == 0) st[b].stale = (j + 1 - st[b].dlen) > nmax + 1;  // the head falls behind while not drafting
  if (acc_out) acc_out[b] = k;
  if (nemit_out) nemit_out[b] = k + 1;
  if (nused_out) nused_out[b] = n;
  if (forced_count == 0) {
    atomicAdd(&cnt->n_target, 1ull);
    atomicAdd(&cnt->n_draft, (unsigned long long)n);
    atomicAdd(&cnt->n_waste, (unsigned long long)(n - k));
    atomicAdd(&cnt->n_tokens, (unsigned long long)(k + 1));
  }
}

// Small state edits used by prefill and force_commit.
__global__ void k_copy_prompt(int *tok, int cap, int b, const int *prompt, int m) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < m; i += gridDim.x * blockDim.x)
    tok[(size_t)b * cap + i] = prompt[i];
}
__global__ void k_finish_prefill(SeqState *st, int *tok, int cap, int b, int m, int chunk, const int *first_tok_slot,
                                 int *user_out) {
  if (threadIdx.x != 0) return;
  const int t = first_tok_slot[0];
  tok[(size_t)b * cap + m] = t;
  st[b].len = m + 1;
  st[b].dlen = m - 1;
  st[b].n = 0; st[b].k_acc = 0; st[b].j_prev = -1; st[b].n_emit = 0; st[b].stale = 0;
  st[b].chunk = chunk;
  if (user_out) *user_out = t;
}
__global__ void k_rewind(SeqState *st, int b, int count, const int *forced_tok, int *draft, int nmax,
                         Counters *cnt) {
  if (threadIdx.x != 0) return;
  const int j = st[b].j_prev;
  if (j < 0) return;
  atomicAdd(&cnt->n_tokens, (unsigned long long)(count - st[b].n_emit));  // wraps correctly for negatives
  st[b].len = j + 1;
  st[b].n = count - 1;
  for (int i = 0; i + 1 < count; ++i) draft[b * nmax + i] = forced_tok[i];
}
__global__ void k_copy_i32(int *dst, const int *src, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = src[i];
}
// Stopping rule of Section 4 (AdaEAGLE-DDD), after draft step `step` (0-based: it produced token step + 1):
// the running log-probability of the draft sequence takes the new token's log-probability; if the predicted
// length is reached (step + 1 >= n) and the sequence is still at or above the threshold, the draft grows by one
// token, within n_max and the cache capacity.  One thread per sequence.
__global__ void k_ddd_update(SeqState *st, const float *lp, float *cum, float thr, int nmax, int cap, int B, int step) {
  const int b = threadIdx.x;
  if (b >= B) return;
  const int n = st[b].n;
  if (n <= step) return;                       // this step did not run for the sequence
  const float c = (step == 0 ? 0.f : cum[b]) + lp[b * nmax + step];
  cum[b] = c;
  const int made = step + 1;
  const int room = cap - st[b].len - 1;        // len + n + 1 <= cap
  if (made >= n && made < nmax && made < room && !(c < thr)) st[b].n = made + 1;
}

// Label pass (Section 3.3 / the draft-length oracle of Section 2.3): full-length drafts for every sequence ...
__global__ void k_set_n_full(SeqState *st, int B, int nmax, int cap) {
  const int b = threadIdx.x;
  if (b >= B) return;
  const int room = cap - st[b].len - 1;
  st[b].n = st[b].len < 2 ? 0 : max(0, min(nmax, room));
}
// ... and, after the verify pass, the length of the longest draft prefix the target confirms.  Nothing is committed.
__global__ void k_label(const SeqState *st, const int *draft, const int *target, int nmax, int B, int *k_out) {
  const int b = threadIdx.x;
  if (b >= B) return;
  const int n = st[b].n;
  int k = 0;
  while (k < n && draft[b * nmax + k] == target[b * (nmax + 1) + k]) ++k;
  k_out[b] = k;
}

// Label collection over start positions (Section 3.3): sequence `seq` is put into the state it had when token j was
// pending (len = j + 1; the draft head's rows of true features up to dlen), with a full-length draft ahead; every
// other sequence of the batch sits the pass out.
__global__ void k_label_begin(SeqState *st, int seq, int B, int len_j, int dlen_j, int nmax, int cap) {
  const int b = threadIdx.x;
  if (b >= B) return;
  if (b != seq) { st[b].n = 0; return; }
  st[b].len = len_j;
  st[b].dlen = dlen_j;
  st[b].j_prev = -1;
  st[b].n = max(0, min(nmax, cap - len_j - 1));
}
// ... the label of that start position (and, optionally, the drafts and the target's choices it came from) ...
__global__ void k_label_one(const SeqState *st, const int *draft, const int *target, int nmax, int seq, int *k_out,
                            int *draft_out, int *target_out) {
  if (threadIdx.x != 0) return;
  const int n = st[seq].n;
  int k = 0;
  while (k < n && draft[seq * nmax + k] == target[seq * (nmax + 1) + k]) ++k;
  *k_out = k;
  for (int i = 0; i < nmax; ++i) {
    if (draft_out) draft_out[i] = i < n ? draft[seq * nmax + i] : -1;
  }
  for (int i = 0; i <= nmax; ++i) {
    if (target_out) target_out[i] = i <= n ? target[seq * (nmax + 1) + i] : -1;
  }
}
// ... and the sequence's own state back (the cache rows and features past the first start position are recomputed
// by the caller's chunk passes).
__global__ void k_label_end(SeqState *st, int seq, int len0, int dlen0, int n0, int j_prev0) {
  if (threadIdx.x != 0) return;
  st[seq].len = len0;
  st[seq].dlen = dlen0;
  st[seq].n = n0;
  st[seq].j_prev = j_prev0;
}

__global__ void k_gather_n(const SeqState *st, int *out, int B) {
  if (threadIdx.x < B) out[threadIdx.x] = st[threadIdx.x].n;
}

}  // namespace ada
