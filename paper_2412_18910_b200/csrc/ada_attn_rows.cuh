// Attention of the multi-row path (ragged batches, prompt chunks) on mma.sync: the rows of one sequence for one
// head over one split of the cache, 16 query rows per CTA (row groups of a long pass across grid.z).
//
// Row r (absolute position pos0 + r) sees cache positions 0 .. pos0 + r: the whole history and the earlier rows
// of its own block (every row's key and value are in the cache before this kernel runs).  The size of a sequence's
// cache splits is fixed when its prompt is read (a quarter of the prompt and its expected continuation, at least an
// eighth of the capacity), so the split a key falls in does not depend on the pass, and a short context is not cut
// into slivers that cost more to set up and merge than to compute.  A warp takes 32-key blocks of the split, in halves
// of 16 keys: one bulk copy brings a half's key rows and one its value rows (they are contiguous in the cache page)
// into one of the warp's two buffers, so the next half is in flight while this one is computed -- scores = q k^T
// as m16n8k16 products per 16 channels, online softmax on the accumulator fragments, weighted values as m16n8k8
// products per 8 channels, 8 keys at a time.  Cache elements are 16-bit halves and enter the products as they are;
// q and the softmax weights are fp32 and enter as a (hi, lo) pair of halves, so each product is issued twice and
// the sums are fp32 (error 2^-22 relative).  Key rows are kept in the cache with their 16-byte chunks XORed by
// (slot & 7), which makes ldmatrix of 8 consecutive keys conflict-free and lets the copy be verbatim.  A copy always
// takes 16 whole rows: rows past the sequence are masked out of the softmax, and every cache row is finite (the
// pools are cleared at initialisation), so they add exact zeros.
// Partial (m, l, o[hd]) per (head, split, row) goes to `part`; k_attn_combine merges the splits in split order.
#pragma once
#include "ada_pass.cuh"

namespace ada {

constexpr int kAttnHalf = 16;   // keys per copy

template <int HD>
constexpr int attn_rows_smem_bytes() {
  return 2 * kRowGroup * HD * 2 + 4 * 2 * 2 * kAttnHalf * HD * 2 + 2 * 4 * kRowGroup * 4 + 4 * 2 * 8;
}

template <int HD>
__global__ void __launch_bounds__(128) k_attn_rows(const Pass *pass, const float *q, const __nv_bfloat16 *kpool,
                                                   const __nv_bfloat16 *vpool, const int *page_table, int pages_per_seq,
                                                   int page_size, int L, int layer, int H, float *part, int nrg,
                                                   int cap, Counters *cnt) {
  static_assert(HD == 64 || HD == 128, "head width");
  constexpr int CH = HD / 8;   // 16-byte chunks per row
  // grid.z = sequences x nrg: CTA (b, rgi) takes the row groups rgi, rgi + nrg, ... of sequence b
  const int hh = blockIdx.x, split = blockIdx.y, b = blockIdx.z / nrg, rgi = blockIdx.z - b * nrg;
  const int R = pass->seq_rows[b];
  if (pass->T <= 0 || R <= 0) return;
  const int row0 = pass->seq_row0[b];
  const int pos0 = pass->row_pos[row0];
  const int nkeys = pos0 + R;
  const int chunk = attn_rows_chunk(pass->seq_chunk[b], cap);
  const int kbeg = split * chunk, kend = min(nkeys, kbeg + chunk);
  if (kbeg >= nkeys) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = H * HD;

  extern __shared__ __align__(128) unsigned char attn_rows_smem[];
  __half *qh_s = reinterpret_cast<__half *>(attn_rows_smem);          // q hi [16][HD], chunks XORed with row & 7
  __half *ql_s = qh_s + kRowGroup * HD;                               // q lo, same layout
  __nv_bfloat16 *stg = reinterpret_cast<__nv_bfloat16 *>(ql_s + kRowGroup * HD);   // [4 warps][2 buffers][K, V][16 keys][HD]
  __nv_bfloat16 *wst = stg + (size_t)warp * 2 * 2 * kAttnHalf * HD;
  float (*o_s)[kRowGroup][HD] = reinterpret_cast<float (*)[kRowGroup][HD]>(stg);    // merge area, over the staging areas
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

  for (int rg = rgi * kRowGroup; rg < R; rg += nrg * kRowGroup) {
    const int nr = min(kRowGroup, R - rg);
    __syncthreads();   // the previous group's merge has read the shared areas; the barriers are initialised
    const int last_pos = pos0 + rg + nr - 1;   // the last position any row of the group sees
    // half h of this warp: keys key0(h) .. key0(h) + 15
    auto key0_of = [&](int h) { return kbeg + 32 * (warp + 4 * (h >> 1)) + kAttnHalf * (h & 1); };
    auto valid = [&](int h) { const int k0 = key0_of(h); return k0 < kend && k0 <= last_pos; };
    auto issue = [&](int h) {   // one lane: the half's key rows and value rows into buffer h & 1
      const int k0 = key0_of(h);
      const int page = page_table[b * pages_per_seq + k0 / page_size];
      const size_t off = (size_t)page * page_stride + head_off + (size_t)(k0 % page_size) * HD;
      __nv_bfloat16 *kst = wst + (size_t)(h & 1) * 2 * kAttnHalf * HD;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic accesses to the buffer come first
      mbar_expect_tx(&bars[h & 1], (unsigned)(2 * kAttnHalf * HD * 2));
      bulk_g2s(kst, kpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1]);
      bulk_g2s(kst + kAttnHalf * HD, vpool + off, (unsigned)(kAttnHalf * HD * 2), &bars[h & 1]);
    };
    if (lane == 0 && valid(0)) issue(0);   // flies under the staging of q
    {   // the group's query rows as (hi, lo) halves; rows past nr are zero
      constexpr int PER = kRowGroup * HD / 4 / 128;
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
        *reinterpret_cast<uint2 *>(ql_s + o) = pl;
      }
    }
    __syncthreads();

    // running maxima, sums and outputs of rows g8r and g8r + 8 over this warp's keys
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[CH][4];
#pragma unroll
    for (int nt = 0; nt < CH; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    const int qp0 = pos0 + rg + g8r, qp1 = qp0 + 8;

    for (int h = 0; valid(h); ++h) {
      if (lane == 0 && valid(h + 1)) issue(h + 1);   // the other buffer: every lane left it at the end of the last turn
      const __nv_bfloat16 *kst = wst + (size_t)(h & 1) * 2 * kAttnHalf * HD, *vst = kst + kAttnHalf * HD;
      mbar_wait(&bars[h & 1], (uses[h & 1]++) & 1u, cnt, &abort_s);
      const int kb = key0_of(h);
#pragma unroll
      for (int sub = 0; sub < 2; ++sub) {
        const int key0 = kb + 8 * sub;          // first of these 8 keys
        if (key0 >= kend || key0 > last_pos) break;
        // ---- scores: 16 rows x 8 keys
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t krow = smem_u32(kst + (size_t)(8 * sub + (lane & 7)) * HD);
        const int ksw = lane & 7;               // = slot & 7: halves start at multiples of 16
        const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int kp = 0; kp < HD / 32; ++kp) {    // pairs of 16-channel steps
          uint32_t kb0, kb1, kb2, kb3;
          ldmatrix_x4(krow + (((kp * 4 + (lane >> 3)) ^ ksw) << 4), kb0, kb1, kb2, kb3);
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const int ks = kp * 2 + h2;
            const uint32_t aoff = (uint32_t)(arow * (HD * 2) + (((ks * 2 + (lane >> 4)) ^ (arow & 7)) << 4));
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(qh_u + aoff, a0, a1, a2, a3);
            mma_f16_k16(sc, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
            ldmatrix_x4(ql_u + aoff, a0, a1, a2, a3);
            mma_f16_k16(sc, a0, a1, a2, a3, h2 ? kb2 : kb0, h2 ? kb3 : kb1);
          }
        }
        // ---- online softmax: this thread holds keys kc, kc + 1 of rows g8r and g8r + 8
        const int kc = key0 + 2 * t4;
        const bool s00 = kc < kend && kc <= qp0, s01 = kc + 1 < kend && kc + 1 <= qp0;
        const bool s10 = kc < kend && kc <= qp1, s11 = kc + 1 < kend && kc + 1 <= qp1;
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
        const uint32_t vrow = smem_u32(vst + (size_t)(8 * sub + (lane & 7)) * HD);
#pragma unroll
        for (int nq = 0; nq < HD / 32; ++nq) {      // four 8-channel tiles per load
          uint32_t v0, v1, v2, v3;
          ldmatrix_x4_trans(vrow + ((nq * 4 + (lane >> 3)) << 4), v0, v1, v2, v3);
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
      __syncwarp();   // every lane is done with this buffer
    }

    // per-warp partials -> shared (over the staging areas, once every warp has left them), merged in warp order
    __syncthreads();
#pragma unroll
    for (int nt = 0; nt < CH; ++nt) {
      *reinterpret_cast<float2 *>(&o_s[warp][g8r][nt * 8 + 2 * t4]) = make_float2(o[nt][0], o[nt][1]);
      *reinterpret_cast<float2 *>(&o_s[warp][g8r + 8][nt * 8 + 2 * t4]) = make_float2(o[nt][2], o[nt][3]);
    }
    if (t4 == 0) {
      m_s[warp][g8r] = m0; l_s[warp][g8r] = l0;
      m_s[warp][g8r + 8] = m1; l_s[warp][g8r + 8] = l1;
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
