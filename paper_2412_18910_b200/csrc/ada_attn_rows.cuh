// Attention of the multi-row path (ragged batches, prompt chunks) on mma.sync: a group of query rows of one sequence
// for one head over one split of the cache per CTA (the row groups of a pass across grid.z).
//
// Row r (absolute position pos0 + r) sees cache positions 0 .. pos0 + r: the whole history and the earlier rows
// of its own block (every row's key and value are in the cache before this kernel runs).  The size of a sequence's
// cache splits is fixed when its prompt is read (the prompt and its expected continuation cut into at most four, at
// least an eighth of the capacity), so the split a key falls in does not depend on the pass, and a short context is not
// cut into slivers that cost more to set up and merge than to compute.  The split's 16-key halves are dealt to the four
// warps in turn: one bulk copy brings a half's key rows and one its value rows (they are contiguous in the cache page)
// into one of the warp's two buffers, so the next half is in flight while this one is computed -- scores = q k^T as
// m16n8k16 products per 16 channels (two tiles of 8 keys), online softmax on the accumulator fragments, weighted values
// as m16n8k16 products over the 16 keys per 8 channels.  Cache elements are 16-bit halves and enter the products as
// they are; q and the softmax weights are fp32 and enter as a (hi, lo) pair of halves, the sums are fp32 (error 2^-22
// relative).  Two forms (template parameter PACK):
//   PACK = false  16 query rows per group; every product is issued twice, for the hi and for the lo halves (prompt
//                 chunks)
//   PACK = true   8 query rows per group: tile rows 0..7 hold their hi halves, rows 8..15 their lo halves, so one
//                 product yields both parts and half as many products and q loads are issued per key (decode passes of
//                 a batch, at most n_max + 1 rows per sequence; every decode row goes through this form whatever the
//                 shape of its pass, so a row's sums do not depend on the pass)
// Key and value rows are kept in the cache with their 16-byte chunks XORed by (slot & 7), which makes ldmatrix of 8
// consecutive keys (plain or transposed) conflict-free and lets the copy be verbatim.  A copy always takes 16 whole
// rows: rows past the sequence are masked out of the softmax, and every cache row is finite (the pools are cleared at
// initialisation), so they add exact zeros.
// Partial (m, l, o[hd]) per (head, split, row) goes to `part`; k_attn_combine merges the splits in split order.
#pragma once
#include "ada_pass.cuh"

namespace ada {

constexpr int kAttnHalf = 16;   // keys per copy

template <int HD>
constexpr int attn_rows_smem_bytes() {
  return 2 * kRowGroup * HD * 2 + 4 * 2 * 2 * kAttnHalf * HD * 2 + 2 * 4 * kRowGroup * 4 + 4 * 2 * 8;
}

template <int HD, bool PACK>
__global__ void __launch_bounds__(128) k_attn_rows(const Pass *pass, const float *q, const __nv_bfloat16 *kpool,
                                                   const __nv_bfloat16 *vpool, const int *page_table, int pages_per_seq,
                                                   int /*page_size = kPageSize*/, int L, int layer, int H, float *part, int nrg,
                                                   int cap, Counters *cnt) {
  static_assert(HD == 64 || HD == 128, "head width");
  constexpr int page_size = kPageSize;
  pdl_launch_dependents();
  pdl_wait();                  // queries and the new cache rows come from the kernel before this one
  constexpr int CH = HD / 8;   // 16-byte chunks per row
  constexpr int RG = PACK ? 8 : kRowGroup;   // query rows per group
  // grid.z = sequences x nrg: CTA (b, rgi) takes the row groups rgi, rgi + nrg, ... of sequence b
  const int hh = blockIdx.x, split = blockIdx.y, b = blockIdx.z / nrg, rgi = blockIdx.z - b * nrg;
  const int4 si = pass->seq_info[b];   // (first row, rows, split size, first position) in one load
  const int row0 = si.x, R = si.y, pos0 = si.w;
  if (R <= 0) return;
  const int nkeys = pos0 + R;
  const int chunk = attn_rows_chunk(si.z, cap);
  const int kbeg = split * chunk, kend = min(nkeys, kbeg + chunk);
  if (kbeg >= nkeys) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = H * HD;

  extern __shared__ __align__(128) unsigned char attn_rows_smem[];
  __half *qh_s = reinterpret_cast<__half *>(attn_rows_smem);          // q hi [16][HD], chunks XORed with row & 7
  __half *ql_s = qh_s + kRowGroup * HD;                               // q lo, same layout
  __nv_bfloat16 *stg = reinterpret_cast<__nv_bfloat16 *>(ql_s + kRowGroup * HD);   // [4 warps][2 buffers][K, V][16 keys][HD]
  __nv_bfloat16 *wst = stg + (size_t)warp * 2 * 2 * kAttnHalf * HD;
  float (*o_s)[kRowGroup][HD + 8] = reinterpret_cast<float (*)[kRowGroup][HD + 8]>(stg);   // merge area, over the staging areas (rows padded: the fragment stores of 8 rows fall into different banks)
  unsigned char *tail = attn_rows_smem + 2 * kRowGroup * HD * 2 + 4 * 2 * 2 * kAttnHalf * HD * 2;
  float (*m_s)[kRowGroup] = reinterpret_cast<float (*)[kRowGroup]>(tail);
  float (*l_s)[kRowGroup] = m_s + 4;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tail + 2 * 4 * kRowGroup * 4) + warp * 2;   // this warp's two buffers
  __shared__ int abort_s;
  const int g8r = lane >> 2, t4 = lane & 3;
  const uint32_t qh_u = smem_u32(qh_s), ql_u = smem_u32(ql_s);
  if (threadIdx.x == 0) abort_s = 0;
  if (lane == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  unsigned uses[2] = {0, 0};   // completed phases of the two buffers' barriers
  const size_t head_off = ((size_t)layer * H + hh) * page_size * HD;   // inside a page: [layer][head][slot][HD]
  const size_t page_stride = (size_t)L * H * page_size * HD;

  for (int rg = rgi * RG; rg < R; rg += nrg * RG) {
    const int nr = min(RG, R - rg);
    __syncthreads();   // the previous group's merge has read the shared areas; the barriers are initialised
    const int last_pos = pos0 + rg + nr - 1;   // the last position any row of the group sees
    // half h of this warp: keys key0(h) .. key0(h) + 15 (the split's halves are dealt to the four warps in turn)
    auto key0_of = [&](int h) { return kbeg + kAttnHalf * (warp + 4 * h); };
    auto valid = [&](int h) { const int k0 = key0_of(h); return k0 < kend && k0 <= last_pos; };
    // cache pages of the warp's halves 32 i + lane, fetched 32 at a time so that no copy waits for a table lookup
    int pages = valid(lane) ? page_table[b * pages_per_seq + key0_of(lane) / page_size] : 0;
    auto issue = [&](int h, int page) {   // one lane: the half's key rows and value rows into buffer h & 1
      const int k0 = key0_of(h);
      const size_t off = (size_t)page * page_stride + head_off + (size_t)(k0 % page_size) * HD;
      __nv_bfloat16 *kst = wst + (size_t)(h & 1) * 2 * kAttnHalf * HD;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic accesses to the buffer come first
      mbar_expect_tx(&bars[h & 1], (unsigned)(2 * kAttnHalf * HD * 2));
      if constexpr (PACK) {   // a decode pass reads a sequence's cache rows once: evict-first in level 2
        bulk_g2s_hint(kst, kpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1], l2_policy_evict_first());
        bulk_g2s_hint(kst + kAttnHalf * HD, vpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1], l2_policy_evict_first());
      } else {                // a prompt chunk's row groups read the same rows again
        bulk_g2s(kst, kpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1]);
        bulk_g2s(kst + kAttnHalf * HD, vpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1]);
      }
    };
    {   // both buffers are free: the first two halves fly under the staging of q
      const int p0 = __shfl_sync(0xffffffffu, pages, 0), p1 = __shfl_sync(0xffffffffu, pages, 1);
      if (lane == 0 && valid(0)) issue(0, p0);
      if (lane == 0 && valid(1)) issue(1, p1);
    }
    {   // the group's query rows as (hi, lo) halves; rows past nr are zero.  PACK: hi of row r in tile row r, lo in row r + 8
      constexpr int PER = RG * HD / 4 / 128;
      float4 qv[PER];
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        const int i = threadIdx.x + u * 128, r = i / (HD / 4), c4 = i - r * (HD / 4);
        qv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < nr) qv[u] = *reinterpret_cast<const float4 *>(q + (size_t)(row0 + rg + r) * d + hh * HD + 4 * c4);
      }
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        const int i = threadIdx.x + u * 128, r = i / (HD / 4), c = 4 * (i - r * (HD / 4));
        const float v[4] = {qv[u].x, qv[u].y, qv[u].z, qv[u].w};
        __half h[4], l[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          h[e] = __float2half_rn(v[e]);
          l[e] = __float2half_rn(v[e] - __half2float(h[e]));
        }
        const int o = r * HD + ((((c >> 3) ^ (r & 7)) << 3) | (c & 7));
        uint2 ph, pl;
        ph.x = (uint32_t)__half_as_ushort(h[0]) | ((uint32_t)__half_as_ushort(h[1]) << 16);
        ph.y = (uint32_t)__half_as_ushort(h[2]) | ((uint32_t)__half_as_ushort(h[3]) << 16);
        pl.x = (uint32_t)__half_as_ushort(l[0]) | ((uint32_t)__half_as_ushort(l[1]) << 16);
        pl.y = (uint32_t)__half_as_ushort(l[2]) | ((uint32_t)__half_as_ushort(l[3]) << 16);
        *reinterpret_cast<uint2 *>(qh_s + o) = ph;
        *reinterpret_cast<uint2 *>((PACK ? qh_s + 8 * HD : ql_s) + o) = pl;
      }
    }
    __syncthreads();

    // running maxima, sums and outputs of rows g8r and g8r + 8 over this warp's keys
    float m0 = -INFINITY, l0 = 0.f;
    [[maybe_unused]] float m1 = -INFINITY, l1 = 0.f;
    float o[CH][4];
#pragma unroll
    for (int nt = 0; nt < CH; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    const int qp0 = pos0 + rg + g8r;
    [[maybe_unused]] const int qp1 = qp0 + 8;

    for (int h = 0; valid(h); ++h) {
      const __nv_bfloat16 *kst = wst + (size_t)(h & 1) * 2 * kAttnHalf * HD, *vst = kst + kAttnHalf * HD;
      mbar_wait(&bars[h & 1], (uses[h & 1]++) & 1u, cnt, &abort_s);
      const int key0 = key0_of(h);            // first of these 16 keys
      if constexpr (PACK) {
        // ---- 8 query rows: tile row r holds the hi half of row r, tile row r + 8 its lo half, so one product gives
        // both parts; this thread's row is g8r, its hi sums are accumulator elements 0, 1 and its lo sums 2, 3
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t krow = smem_u32(kst + (size_t)(lane & 7) * HD);
        const int ksw = lane & 7;
        const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int kp = 0; kp < HD / 32; ++kp) {
          uint32_t ka0, ka1, ka2, ka3, kb0, kb1, kb2, kb3;
          const uint32_t koff = (uint32_t)(((kp * 4 + (lane >> 3)) ^ ksw) << 4);
          ldmatrix_x4(krow + koff, ka0, ka1, ka2, ka3);
          ldmatrix_x4(krow + 8 * HD * 2 + koff, kb0, kb1, kb2, kb3);
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const int ks = kp * 2 + h2;
            const uint32_t aoff = (uint32_t)(arow * (HD * 2) + (((ks * 2 + (lane >> 4)) ^ (arow & 7)) << 4));
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(qh_u + aoff, a0, a1, a2, a3);
            mma_f16_k16(sa, a0, a1, a2, a3, h2 ? ka2 : ka0, h2 ? ka3 : ka1);
            mma_f16_k16(sb, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
          }
        }
        // ---- online softmax of row g8r: keys kc, kc + 1, kc + 8, kc + 9
        const int kc = key0 + 2 * t4;
        const float s0[4] = {sa[0] + sa[2], sa[1] + sa[3], sb[0] + sb[2], sb[1] + sb[3]};
        float p0[4] = {0.f, 0.f, 0.f, 0.f}, c0 = 1.f, mn0;
        if (key0 + kAttnHalf <= kend && key0 + kAttnHalf - 1 <= pos0 + rg) {   // every row sees all 16 keys (warp-uniform)
          float mx0 = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s0[2], s0[3]));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
          mn0 = fmaxf(m0, mx0);
#pragma unroll
          for (int j = 0; j < 4; ++j) p0[j] = __expf(s0[j] - mn0);
          c0 = __expf(m0 - mn0);
        } else {
          bool ok0[4];
          float mx0 = -INFINITY;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int k = kc + (j & 1) + 8 * (j >> 1);
            ok0[j] = k < kend && k <= qp0;
            mx0 = fmaxf(mx0, ok0[j] ? s0[j] : -INFINITY);
          }
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
          mn0 = fmaxf(m0, mx0);
          if (mn0 > -INFINITY) {
#pragma unroll
            for (int j = 0; j < 4; ++j) p0[j] = ok0[j] ? __expf(s0[j] - mn0) : 0.f;
            c0 = __expf(m0 - mn0);
          }
        }
        float ps0 = (p0[0] + p0[1]) + (p0[2] + p0[3]);
        ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1);
        ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2);
        l0 = l0 * c0 + ps0;
        m0 = mn0;
        // weights: A operand rows g8r (hi halves) and g8r + 8 (lo halves); a0, a1: keys 0..7, a2, a3: keys 8..15
        uint32_t aw[4];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const __half2 ph = __floats2half2_rn(p0[2 * j], p0[2 * j + 1]);
          const float2 pf = __half22float2(ph);
          const __half2 pl = __floats2half2_rn(p0[2 * j] - pf.x, p0[2 * j + 1] - pf.y);
          aw[2 * j] = *reinterpret_cast<const uint32_t *>(&ph);
          aw[2 * j + 1] = *reinterpret_cast<const uint32_t *>(&pl);
        }
        // ---- values: elements 0, 1 of a tile collect the hi weights' sums of row g8r, elements 2, 3 the lo weights' sums
        const uint32_t vrow = smem_u32(vst + (size_t)((lane & 7) + 8 * ((lane >> 3) & 1)) * HD);
        if (__any_sync(0xffffffffu, c0 != 1.f)) {
#pragma unroll
          for (int nt = 0; nt < CH; ++nt) { o[nt][0] *= c0; o[nt][1] *= c0; o[nt][2] *= c0; o[nt][3] *= c0; }
        }
#pragma unroll
        for (int c2 = 0; c2 < HD / 16; ++c2) {
          uint32_t v0, v1, v2, v3;
          ldmatrix_x4_trans(vrow + (((2 * c2 + (lane >> 4)) ^ (lane & 7)) << 4), v0, v1, v2, v3);
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(o[2 * c2]), aw[0], aw[1], aw[2], aw[3], v0, v1);
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(o[2 * c2 + 1]), aw[0], aw[1], aw[2], aw[3], v2, v3);
        }
      } else {
        // ---- scores: 16 rows x 16 keys as two tiles of 8 keys (sa: keys 0..7, sb: keys 8..15)
        // (the hi and the lo products have accumulators of their own, added at the end: four chains of 8 products)
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        float sal[4] = {0.f, 0.f, 0.f, 0.f}, sbl[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t krow = smem_u32(kst + (size_t)(lane & 7) * HD);
        const int ksw = lane & 7;               // = slot & 7: halves start at multiples of 16
        const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int kp = 0; kp < HD / 32; ++kp) {    // pairs of 16-channel steps
          uint32_t ka0, ka1, ka2, ka3, kb0, kb1, kb2, kb3;
          const uint32_t koff = (uint32_t)(((kp * 4 + (lane >> 3)) ^ ksw) << 4);
          ldmatrix_x4(krow + koff, ka0, ka1, ka2, ka3);
          ldmatrix_x4(krow + 8 * HD * 2 + koff, kb0, kb1, kb2, kb3);
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const int ks = kp * 2 + h2;
            const uint32_t aoff = (uint32_t)(arow * (HD * 2) + (((ks * 2 + (lane >> 4)) ^ (arow & 7)) << 4));
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(qh_u + aoff, a0, a1, a2, a3);
            mma_f16_k16(sa, a0, a1, a2, a3, h2 ? ka2 : ka0, h2 ? ka3 : ka1);
            mma_f16_k16(sb, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
            ldmatrix_x4(ql_u + aoff, a0, a1, a2, a3);
            mma_f16_k16(sal, a0, a1, a2, a3, h2 ? ka2 : ka0, h2 ? ka3 : ka1);
            mma_f16_k16(sbl, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) { sa[j] += sal[j]; sb[j] += sbl[j]; }
        // ---- online softmax: this thread holds keys kc, kc + 1, kc + 8, kc + 9 of rows g8r and g8r + 8
        const int kc = key0 + 2 * t4;
        const float s0[4] = {sa[0], sa[1], sb[0], sb[1]}, s1[4] = {sa[2], sa[3], sb[2], sb[3]};
        float p0[4] = {0.f, 0.f, 0.f, 0.f}, p1[4] = {0.f, 0.f, 0.f, 0.f}, c0 = 1.f, c1 = 1.f;
        float mn0, mn1;
        if (key0 + kAttnHalf <= kend && key0 + kAttnHalf - 1 <= pos0 + rg) {
          // every row of the group sees all 16 keys (warp-uniform): no masks
          float mx0 = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s0[2], s0[3])), mx1 = fmaxf(fmaxf(s1[0], s1[1]), fmaxf(s1[2], s1[3]));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
          mn0 = fmaxf(m0, mx0); mn1 = fmaxf(m1, mx1);
#pragma unroll
          for (int j = 0; j < 4; ++j) { p0[j] = __expf(s0[j] - mn0); p1[j] = __expf(s1[j] - mn1); }
          c0 = __expf(m0 - mn0); c1 = __expf(m1 - mn1);
        } else {
          bool ok0[4], ok1[4];    // [key slot] for row g8r / g8r + 8
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int k = kc + (j & 1) + 8 * (j >> 1);
            ok0[j] = k < kend && k <= qp0;
            ok1[j] = k < kend && k <= qp1;
          }
          float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            mx0 = fmaxf(mx0, ok0[j] ? s0[j] : -INFINITY);
            mx1 = fmaxf(mx1, ok1[j] ? s1[j] : -INFINITY);
          }
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
          mn0 = fmaxf(m0, mx0); mn1 = fmaxf(m1, mx1);
          if (mn0 > -INFINITY) {
#pragma unroll
            for (int j = 0; j < 4; ++j) p0[j] = ok0[j] ? __expf(s0[j] - mn0) : 0.f;
            c0 = __expf(m0 - mn0);
          }
          if (mn1 > -INFINITY) {
#pragma unroll
            for (int j = 0; j < 4; ++j) p1[j] = ok1[j] ? __expf(s1[j] - mn1) : 0.f;
            c1 = __expf(m1 - mn1);
          }
        }
        float ps0 = (p0[0] + p0[1]) + (p0[2] + p0[3]), ps1 = (p1[0] + p1[1]) + (p1[2] + p1[3]);
        ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1); ps1 += __shfl_xor_sync(0xffffffffu, ps1, 1);
        ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2); ps1 += __shfl_xor_sync(0xffffffffu, ps1, 2);
        l0 = l0 * c0 + ps0; l1 = l1 * c1 + ps1;
        m0 = mn0; m1 = mn1;
        // weights as (hi, lo) halves: A operand of a k = 16 product: a0 = row g8r keys 0..7, a1 = row g8r + 8 keys 0..7,
        // a2 = row g8r keys 8..15, a3 = row g8r + 8 keys 8..15 (this thread's pair of each)
        uint32_t ah[4], al[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float x = (j & 1) ? p1[2 * (j >> 1)] : p0[2 * (j >> 1)], y = (j & 1) ? p1[2 * (j >> 1) + 1] : p0[2 * (j >> 1) + 1];
          const __half2 ph = __floats2half2_rn(x, y);
          const float2 pf = __half22float2(ph);
          const __half2 pl = __floats2half2_rn(x - pf.x, y - pf.y);
          ah[j] = *reinterpret_cast<const uint32_t *>(&ph);
          al[j] = *reinterpret_cast<const uint32_t *>(&pl);
        }
        // ---- values: out[16 rows][HD] += w[16 x 16 keys] v[16 keys x HD], two 8-channel tiles per load
        const uint32_t vrow = smem_u32(vst + (size_t)((lane & 7) + 8 * ((lane >> 3) & 1)) * HD);
        if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {   // some running maximum moved: rescale the sums so far
#pragma unroll
          for (int nt = 0; nt < CH; ++nt) { o[nt][0] *= c0; o[nt][1] *= c0; o[nt][2] *= c1; o[nt][3] *= c1; }
        }
#pragma unroll
        for (int c2 = 0; c2 < HD / 16; ++c2) {
          uint32_t v0, v1, v2, v3;   // (keys 0..7, keys 8..15) of channel tile 2 c2, then of tile 2 c2 + 1
          ldmatrix_x4_trans(vrow + (((2 * c2 + (lane >> 4)) ^ (lane & 7)) << 4), v0, v1, v2, v3);
          float *oa = o[2 * c2], *ob = o[2 * c2 + 1];
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(oa), ah[0], ah[1], ah[2], ah[3], v0, v1);
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(oa), al[0], al[1], al[2], al[3], v0, v1);
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(ob), ah[0], ah[1], ah[2], ah[3], v2, v3);
          mma_f16_k16(*reinterpret_cast<float (*)[4]>(ob), al[0], al[1], al[2], al[3], v2, v3);
        }
      }
      __syncwarp();   // every lane is done with this buffer: the half after the next one goes into it
      if (((h + 2) & 31) == 0) pages = valid(h + 2 + lane) ? page_table[b * pages_per_seq + key0_of(h + 2 + lane) / page_size] : 0;
      const int pnext = __shfl_sync(0xffffffffu, pages, (h + 2) & 31);
      if (lane == 0 && valid(h + 2)) issue(h + 2, pnext);
    }

    // per-warp partials -> shared (over the staging areas, once every warp has left them), merged in warp order
    __syncthreads();
#pragma unroll
    for (int nt = 0; nt < CH; ++nt) {
      if constexpr (PACK) {   // hi and lo sums of the row
        *reinterpret_cast<float2 *>(&o_s[warp][g8r][nt * 8 + 2 * t4]) = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
      } else {
        *reinterpret_cast<float2 *>(&o_s[warp][g8r][nt * 8 + 2 * t4]) = make_float2(o[nt][0], o[nt][1]);
        *reinterpret_cast<float2 *>(&o_s[warp][g8r + 8][nt * 8 + 2 * t4]) = make_float2(o[nt][2], o[nt][3]);
      }
    }
    if (t4 == 0) {
      m_s[warp][g8r] = m0; l_s[warp][g8r] = l0;
      if constexpr (!PACK) { m_s[warp][g8r + 8] = m1; l_s[warp][g8r + 8] = l1; }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < nr * HD; i += 128) {
      const int r = i / HD, c = i - r * HD;
      float M = m_s[0][r];
      for (int w = 1; w < 4; ++w) M = fmaxf(M, m_s[w][r]);
      float lo = 0.f, oo = 0.f;
      if (M > -INFINITY) {
        for (int w = 0; w < 4; ++w) {
          const float e = __expf(m_s[w][r] - M);
          lo += l_s[w][r] * e;
          oo += o_s[w][r][c] * e;
        }
      }
      float *pp = part + (((size_t)hh * kAttnSplits + split) * kMaxRows + (row0 + rg + r)) * (HD + 2);
      pp[c] = oo;
      if (c == 0) { pp[HD] = M; pp[HD + 1] = lo; }
    }
  }
}

}  // namespace ada
