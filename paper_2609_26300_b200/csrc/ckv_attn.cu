// Exact attention over a list of cache pages (split along the list), the removal of the selected
// blocks' mean-compensation terms, and the final log-sum-exp merge (Eq. 12).
//
// Sparse mode: the page list of a unit is the pages of its selected blocks, in position order.
// Dense mode: every page of the sequence (Eq. 12 with S = all blocks; Sec. 3.1).
//
// A CTA takes a contiguous slice of the list; each of its 8 warps takes every 8th page.  Within a
// warp a token row (128 elements) is spread over the 16 lanes of a half warp (8 coordinates per
// lane, one 16-byte load for bf16) and the two half warps take alternate rows.  QK^T partial sums
// are reduced across the 16 lanes with a work-sharing shuffle tree, so that each lane ends up
// owning the logits of one row for half of the heads and evaluates those exponentials only; the
// probabilities go through a small shared-memory tile back to the lanes that hold the V rows.
// Running maxima are kept per warp and only raised when exceeded by a slack (the partial
// (m, l, acc) stays an exact representation of sum e^{z} v for any m).
//
// For every selected block the scan kernel has already added the block's mean term
// |b| e^{zbar} vbar_b to the all-block compensation sum; here the same term is subtracted from the
// exact partial, so that  merge = exact(S) + mean(all) - mean(S) = exact(S) + mean(not S).
#include "ckv_internal.cuh"
#include "ckv_pipe.cuh"

namespace {

using namespace ckv_pipe;

constexpr int kMaxBuf = 4;                       // page buffers per warp
constexpr int kPageElems = CKV_PAGE * CKV_D;     // elements of one head's K (or V) page

template <int G, typename T, bool DENSE>
__global__ void __launch_bounds__(256, (DENSE || G > 4) ? 1 : 2)
ckv_attn_kernel(CkvDev P, const T *__restrict__ q, const T *__restrict__ k_pool, const T *__restrict__ v_pool,
                const int *__restrict__ page_table, const int *__restrict__ seq_lens,
                const int *__restrict__ sel_ids, const int *__restrict__ sel_cnt, int kcap, int pages_per_split,
                int nbuf) {
  constexpr int NV = 8 * G;                      // logits per lane before the reduction (8 rows x G heads)
  constexpr int KEEP = (NV >= 16) ? NV / 16 : 1;  // logits per lane after it
  constexpr int HSPLIT = (G >= 2) ? 2 : 1;        // a row's heads are shared by this many lanes
  extern __shared__ __align__(128) unsigned char pg_mem[];   // [8 warps][nbuf][K page | V page]
  __shared__ __align__(8) uint64_t bars[8][kMaxBuf];
  __shared__ int meta[8][kMaxBuf][4];             // physical page (or -1), valid tokens, block id, list index
  __shared__ float sq[G][CKV_D];
  __shared__ __align__(16) float pbuf[8][CKV_PAGE][G];
  __shared__ __align__(16) float red[8][G][CKV_PART_STRIDE];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, hw = lane >> 4, li = lane & 15;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int N = max(min(seq_lens[s], P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) / P.bs;
  const int nsel = DENSE ? X : min(sel_cnt[unit], kcap);
  const int total = DENSE ? (N + CKV_PAGE - 1) / CKV_PAGE : nsel * P.ppb;
  const bool comp = !DENSE && nsel < X && !(P.variant & CKV_VARIANT_DROP);
  const int p0 = blockIdx.x * pages_per_split;
  const int p1 = min(p0 + pages_per_split, total);
  float *part = P.attn_part + ((size_t)unit * CKV_MAX_SPLITS + blockIdx.x) * G * CKV_PART_STRIDE;
  if (p0 >= total) {
    if (tid < G) { part[tid * CKV_PART_STRIDE] = -CUDART_INF_F; part[tid * CKV_PART_STRIDE + 1] = 0.f; }
    return;
  }

  T *wbuf = reinterpret_cast<T *>(pg_mem) + (size_t)warp * nbuf * 2 * kPageElems;
  uint64_t *wbar = bars[warp];
  if (lane == 0) {
    for (int b = 0; b < nbuf; ++b) mbar_init(&wbar[b], 1);
    fence_barrier_init();
  }
  for (int idx = tid; idx < G * CKV_D; idx += 256)
    sq[idx / CKV_D][idx % CKV_D] = to_float(q[((size_t)s * P.Hq + h * G) * CKV_D + idx]) * (P.scale * kLog2e);
  __syncthreads();

  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
  const int pshift = P.ppb == 1 ? 0 : (P.ppb == 2 ? 1 : 2);
  const int n_mine = (p1 - p0 - warp + 7) >> 3;   // this warp's pages: list index p0 + warp + 8 n
  bool bad = false;

  // lane 0: resolve list entry n to a physical page and start its copy into buffer n % nbuf
  auto issue = [&](int n, int b) {
    const int i = p0 + warp + 8 * n;
    int phys = -1, ntok = 0, blk = -1, page = i;
    bool ok = true;
    if (!DENSE) {
      blk = sel_ids[(size_t)unit * kcap + (i >> pshift)];
      ok = blk >= 0 && blk < X;
      if (!ok) blk = -1;
      page = (blk << pshift) + (i & (P.ppb - 1));
    }
    if (ok) {
      ntok = min(CKV_PAGE, N - page * CKV_PAGE);
      if (ntok > 0) {
        phys = pt_row[page];
        if (phys < 0 || phys >= P.num_pages) { phys = -1; bad = true; }
      } else {
        ntok = 0;
      }
    }
    meta[warp][b][0] = phys; meta[warp][b][1] = ntok; meta[warp][b][2] = blk; meta[warp][b][3] = i;
    if (phys >= 0) {
      const uint32_t bytes = (uint32_t)ntok * CKV_D * sizeof(T);
      const size_t src = ((size_t)phys * P.Hkv + h) * kPageElems;
      T *dst = wbuf + (size_t)b * 2 * kPageElems;
      mbar_arrive_expect_tx(&wbar[b], 2 * bytes);
      const uint32_t lo = smem_u32(pg_mem), hi = lo + (uint32_t)(8 * nbuf * 2 * kPageElems * sizeof(T));
      bool ok = bulk_g2s_checked(dst, k_pool + src, bytes, &wbar[b], lo, hi);
      ok = ok && bulk_g2s_checked(dst + kPageElems, v_pool + src, bytes, &wbar[b], lo, hi);
      if (!ok) atomicOr(P.status, CKV_DEV_BAD_COPY);
    }
  };
  int issued = 0;
  if (lane == 0)
    for (; issued < nbuf && issued < n_mine; ++issued) issue(issued, issued);
  __syncwarp();

  float qr[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int i = 0; i < 8; ++i) qr[g][i] = sq[g][8 * li + i];

  float acc[G][8], m_ref[G], m_own[KEEP], l_own[KEEP];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_ref[g] = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;
  }
#pragma unroll
  for (int jj = 0; jj < KEEP; ++jj) { m_own[jj] = -CUDART_INF_F; l_own[jj] = 0.f; }
  // after the reduction this lane owns row (li / 2) of its half warp and heads [g_own0, g_own0 + KEEP)
  const int g_own0 = (G >= 2) ? (li & 1) * KEEP : 0;
  const int t_own = hw + 2 * (li >> 1);
  const float *lz = P.lz + (size_t)unit * P.max_blocks * G;
  const __nv_bfloat16 *vmean = P.vmean + (size_t)unit * P.max_blocks * P.row_elems;
  uint32_t phase_bits = 0;   // bit b: parity of the next completion of buffer b
  bool aborted = false;
  int n_abort = 0;

  for (int n = 0, b = 0; n < n_mine; ++n) {
    const int phys = meta[warp][b][0], ntok = meta[warp][b][1], blk = meta[warp][b][2], i = meta[warp][b][3];
    if (phys >= 0 && !aborted) {
      if (!mbar_wait(&wbar[b], (phase_bits >> b) & 1)) {
        atomicOr(P.status, CKV_DEV_TIMEOUT);
        aborted = true;
      }
      aborted = __any_sync(0xffffffffu, aborted);
      if (aborted) n_abort = n;
    }
    if (phys >= 0 && !aborted) {
      phase_bits ^= 1u << b;
      const T *kp = wbuf + (size_t)b * 2 * kPageElems + 8 * li;
      const T *vp = kp + kPageElems;
      float sv[NV];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        float kf[8];
        load8<false>(kp + t * CKV_D, kf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float z = 0.f;
#pragma unroll
          for (int c = 0; c < 8; ++c) z = fmaf(qr[g][c], kf[c], z);
          sv[j * G + g] = (t < ntok) ? z : 0.f;   // rows past the last token hold stale bytes
        }
      }
      reduce16<NV, KEEP>(sv, li);
      // sv[0..KEEP): logits (log2 units) of row t_own for heads g_own0 + jj
      const bool row_ok = t_own < ntok;
      bool need = false;
#pragma unroll
      for (int jj = 0; jj < KEEP; ++jj) {
        if (!row_ok) sv[jj] = -CUDART_INF_F;
        need |= sv[jj] > m_own[jj] + CKV_RESCALE_SLACK;
      }
      if (__any_sync(0xffffffffu, need)) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float cand = -CUDART_INF_F;
#pragma unroll
          for (int jj = 0; jj < KEEP; ++jj)
            if (g_own0 + jj == g) cand = sv[jj];
          cand = warp_max(cand);
          if (cand > m_ref[g]) {
            const float sc = exp2_diff(m_ref[g], cand);
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[g][c] *= sc;
#pragma unroll
            for (int jj = 0; jj < KEEP; ++jj)
              if (g_own0 + jj == g) { l_own[jj] *= sc; m_own[jj] = cand; }
            m_ref[g] = cand;
          }
        }
      }
      float pr[KEEP];
#pragma unroll
      for (int jj = 0; jj < KEEP; ++jj) {
        pr[jj] = row_ok ? exp2f(sv[jj] - m_own[jj]) : 0.f;
        // with G == 1 two lanes hold the same logit: only the even one counts it
        if (G >= 2 || (li & 1) == 0) l_own[jj] += pr[jj];
      }
      float *prow = &pbuf[warp][t_own][g_own0];
#pragma unroll
      for (int jj = 0; jj < KEEP; ++jj) prow[jj] = pr[jj];
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          const float *pp = pbuf[warp][t];
          float vf[8];
          load8<false>(vp + t * CKV_D, vf);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float pg = pp[g];
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[g][c] = fmaf(pg, vf[c], acc[g][c]);
          }
        }
      }
      if (comp && (i & (P.ppb - 1)) == 0) {
        // take this block's mean term |b| e^{zbar} vbar_b back out (it is part of the all-block sum)
        float zl2[G];
        bool raise = false;
#pragma unroll
        for (int g = 0; g < G; ++g) {
          zl2[g] = __ldg(lz + (size_t)g * P.max_blocks + blk);
          raise |= zl2[g] > m_ref[g] + CKV_RESCALE_SLACK;
        }
        if (raise) {   // warp-uniform: every lane evaluates the same values
#pragma unroll
          for (int g = 0; g < G; ++g) {
            if (zl2[g] > m_ref[g]) {
              const float sc = exp2_diff(m_ref[g], zl2[g]);
#pragma unroll
              for (int c = 0; c < 8; ++c) acc[g][c] *= sc;
#pragma unroll
              for (int jj = 0; jj < KEEP; ++jj)
                if (g_own0 + jj == g) { l_own[jj] *= sc; m_own[jj] = zl2[g]; }
              m_ref[g] = zl2[g];
            }
          }
        }
        if (hw == 0) {
          float vb[8];
          load_split8(vmean + (size_t)blk * P.row_elems, li, blk, vb, P.row_elems == CKV_ROW_ELEMS);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float wbar_g = exp2f(zl2[g] - m_ref[g]);
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[g][c] = fmaf(-wbar_g, vb[c], acc[g][c]);
#pragma unroll
            for (int jj = 0; jj < KEEP; ++jj)
              if (g_own0 + jj == g && li < HSPLIT) l_own[jj] -= wbar_g;
          }
        }
      }
    }
    // the buffer is free: order this warp's shared-memory reads before the next bulk copy into it
    fence_proxy_async();
    __syncwarp();
    if (lane == 0 && !aborted && issued < n_mine) { issue(issued, b); ++issued; }
    __syncwarp();
    if (++b == nbuf) b = 0;
  }
  if (aborted && lane == 0) {
    // leave no bulk copy in flight into this warp's buffers
    for (int n = n_abort; n < issued; ++n) {
      const int b = n % nbuf;
      if (meta[warp][b][0] >= 0) mbar_wait(&wbar[b], (phase_bits >> b) & 1);
    }
  }
  if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);

  // warp totals: both half warps share m_ref, so accumulators add directly
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[g][c] += __shfl_xor_sync(0xffffffffu, acc[g][c], 16);
    float lg = 0.f;
#pragma unroll
    for (int jj = 0; jj < KEEP; ++jj)
      if (g_own0 + jj == g) lg = l_own[jj];
    lg = warp_sum(lg);
    float *r = red[warp][g];
    if (hw == 0) {
      *reinterpret_cast<float4 *>(r + 4 + 8 * li) = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
      *reinterpret_cast<float4 *>(r + 8 + 8 * li) = make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]);
    }
    if (lane == 0) { r[0] = m_ref[g]; r[1] = lg; }
  }
  __syncthreads();
  for (int idx = tid; idx < G * CKV_D; idx += 256) {
    const int g = idx / CKV_D, c = idx % CKV_D;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < 8; ++w) M = fmaxf(M, red[w][g][0]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float sc = exp2_diff(red[w][g][0], M);
      num = fmaf(red[w][g][4 + c], sc, num);
      den = fmaf(red[w][g][1], sc, den);
    }
    part[g * CKV_PART_STRIDE + 4 + c] = num;
    if (c == 0) { part[g * CKV_PART_STRIDE] = M; part[g * CKV_PART_STRIDE + 1] = den; }
  }
}

// out_{g} = sum of all partials under one normaliser (Eq. 12).  One CTA per (sequence, query head),
// one thread per output coordinate.  Partials: the unit's attention splits and, unless every block
// was selected, the unit's scan partials (a contiguous run of entries, recomputed here from the same tile
// arithmetic the scan uses).
constexpr int kMergeMax = CKV_MAX_SPLITS + CKV_MAX_SCAN_CTAS * CKV_SCAN_WARPS + 1;

constexpr int kMergeGroups = 4;   // thread groups of CKV_D threads, each summing every fourth partial

template <typename T>
__global__ void __launch_bounds__(CKV_D *kMergeGroups) ckv_merge_kernel(CkvDev P, const int *__restrict__ seq_lens,
                                                                        const int *__restrict__ sel_cnt, int n_splits,
                                                                        int scan_grid, int units, bool dense,
                                                                        T *__restrict__ out, float *__restrict__ lse) {
  constexpr int NT = CKV_D * kMergeGroups;
  __shared__ float s_scale[kMergeMax];
  __shared__ float s_l[kMergeMax];
  __shared__ const float *s_ptr[kMergeMax];
  __shared__ float s_wmax[NT / 32];
  __shared__ float s_num[kMergeGroups][CKV_D], s_den[kMergeGroups];
  __shared__ int s_cfirst, s_ccount;
  const int hq = blockIdx.x, s = blockIdx.y, tid = threadIdx.x, c = tid % CKV_D, grp = tid / CKV_D;
  const int G = P.G, unit = s * P.Hkv + hq / G, g = hq % G;
  const int N = max(min(seq_lens[s], P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) / P.bs;
  const bool comp = !dense && sel_cnt[unit] < X && !(P.variant & CKV_VARIANT_DROP);
  if (tid < 32) {
    int cfirst = 0, ccount = 0;   // first entry, number of entries
    if (comp) unit_scan_entries(P, CkvClampedLens{seq_lens, P.max_blocks * P.bs}, units, unit, scan_grid, tid, cfirst, ccount);
    if (tid == 0) { s_cfirst = cfirst; s_ccount = ccount; }
  }
  __syncthreads();
  const int n_comp = s_ccount;
  const int n = n_splits + n_comp;
  const size_t step = (size_t)G * CKV_PART_STRIDE;
  const float *ap = P.attn_part + ((size_t)unit * CKV_MAX_SPLITS * G + g) * CKV_PART_STRIDE;
  const float *cp = P.comp_part + ((size_t)s_cfirst * G + g) * CKV_PART_STRIDE;
  float mloc = -CUDART_INF_F;
  for (int i = tid; i < n; i += NT) {
    const float *p = i < n_splits ? ap + (size_t)i * step : cp + (size_t)(i - n_splits) * step;
    const float m = p[0];
    s_ptr[i] = p; s_scale[i] = m; s_l[i] = p[1];
    mloc = fmaxf(mloc, m);
  }
  mloc = warp_max(mloc);
  if ((tid & 31) == 0) s_wmax[tid >> 5] = mloc;
  __syncthreads();
  float M = s_wmax[0];
#pragma unroll
  for (int w = 1; w < NT / 32; ++w) M = fmaxf(M, s_wmax[w]);
  for (int i = tid; i < n; i += NT) s_scale[i] = exp2_diff(s_scale[i], M);
  __syncthreads();
  // group grp sums partials grp, grp + 4, ...; four loads in flight per thread; empty partials are skipped
  float num = 0.f, den = 0.f;
  for (int i = grp; i < n; i += 4 * kMergeGroups) {
    float a[4], sc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int ii = i + k * kMergeGroups;
      sc[k] = ii < n ? s_scale[ii] : 0.f;
      a[k] = sc[k] != 0.f ? s_ptr[ii][4 + c] : 0.f;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int ii = i + k * kMergeGroups;
      num = fmaf(a[k], sc[k], num);
      if (ii < n) den = fmaf(s_l[ii], sc[k], den);
    }
  }
  s_num[grp][c] = num;
  if (c == 0) s_den[grp] = den;
  __syncthreads();
  if (grp == 0) {
#pragma unroll
    for (int k = 1; k < kMergeGroups; ++k) { num += s_num[k][c]; den += s_den[k]; }
    const size_t o = ((size_t)s * P.Hq + hq) * CKV_D + c;
    store_out(out + o, N > 0 ? num / den : 0.f);
    if (lse != nullptr && c == 0) lse[(size_t)s * P.Hq + hq] = N > 0 ? (M + log2f(den)) * kLn2 : -CUDART_INF_F;
  }
}

// Static shared memory of the attention kernel (query tile, probability tile, warp partials, barriers).
inline size_t attn_static_smem(int G) {
  return (size_t)G * CKV_D * 4 + (size_t)8 * CKV_PAGE * G * 4 + (size_t)8 * G * CKV_PART_STRIDE * 4 + 1024;
}
inline size_t attn_page_pair_bytes(const ckv_ctx *c) {
  return (size_t)2 * kPageElems * (c->layout.kv_dtype == CKV_BF16 ? 2 : 4);
}
// Page buffers per warp: one for the sparse list (a warp owns one or two pages), as many as fit (up to 3) for dense.
inline int attn_nbuf(const ckv_ctx *c, bool dense, int pps) {
  const size_t per_buf = 8 * attn_page_pair_bytes(c);
  const size_t room = 220 * 1024 - attn_static_smem(c->dev.G);
  int fit = (int)(room / per_buf);
  if (fit < 1) fit = 1;
  int want = dense ? 3 : (pps > 8 ? 2 : 1);
  return want < fit ? want : fit;
}

template <int G, typename T>
cudaError_t launch_gt(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                      const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt, int kcap,
                      dim3 grid, int pps, cudaStream_t st) {
  const int nbuf = attn_nbuf(c, dense, pps);
  const size_t smem = (size_t)nbuf * 8 * attn_page_pair_bytes(c);
  if (dense)
    ckv_attn_kernel<G, T, true><<<grid, 256, smem, st>>>(c->dev, (const T *)q, (const T *)k_pool, (const T *)v_pool,
                                                          page_table, seq_lens, sel_ids, sel_cnt, kcap, pps, nbuf);
  else
    ckv_attn_kernel<G, T, false><<<grid, 256, smem, st>>>(c->dev, (const T *)q, (const T *)k_pool, (const T *)v_pool,
                                                           page_table, seq_lens, sel_ids, sel_cnt, kcap, pps, nbuf);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                     const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt, int kcap,
                     dim3 grid, int pps, cudaStream_t st) {
  if (c->layout.kv_dtype == CKV_BF16)
    return launch_gt<G, __nv_bfloat16>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap,
                                       grid, pps, st);
  return launch_gt<G, float>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
}

template <int G, typename T>
cudaError_t configure_gt(const ckv_ctx *c) {
  const int smem = (int)(220 * 1024 - attn_static_smem(G));
  cudaError_t e = cudaFuncSetAttribute(ckv_attn_kernel<G, T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(ckv_attn_kernel<G, T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return e;
}
template <int G>
cudaError_t configure_g(const ckv_ctx *c) {
  if (c->layout.kv_dtype == CKV_BF16) return configure_gt<G, __nv_bfloat16>(c);
  return configure_gt<G, float>(c);
}

}  // namespace

// Opt in to the dynamic shared memory this context's attention instantiations need, on the current device.
cudaError_t ckv_configure_attn(const ckv_ctx *c) {
  switch (c->dev.G) {
    case 1: return configure_g<1>(c);
    case 2: return configure_g<2>(c);
    case 4: return configure_g<4>(c);
    case 8: return configure_g<8>(c);
  }
  return cudaErrorInvalidValue;
}

cudaError_t ckv_launch_attn(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                            const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt,
                            int kcap, int batch, int max_len, int scan_grid, void *out, float *lse,
                            int *n_splits_out, bool *merged_out, cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int units = batch * P.Hkv;
  const int xmax = (max_len + P.bs - 1) / P.bs;
  const int total = dense ? (max_len + CKV_PAGE - 1) / CKV_PAGE : min(kcap, xmax) * P.ppb;
  const bool mma = c->layout.kv_dtype == CKV_BF16;
  const int sms = c->sm_count > 0 ? c->sm_count : 148;
  // Splits per unit: the dense pass (and the fp32 kernel) get about four CTAs per SM overall; the tensor-core
  // kernel's sparse mode is sized below.  At most CKV_MAX_SPLITS splits.
  int n_splits = (sms * 4 + units - 1) / units;
  if (dense && mma) {
    // One 8-warp CTA per SM: the grid runs in waves, and a last wave that is mostly empty costs a whole wave's time
    // (19 splits of 32 units = 608 CTAs = 4.1 waves took 352 us; 9 or 18 splits, 1.95 and 3.9 waves, 320 us).  Among
    // 1.5 to 4.2 CTAs per SM, the split count whose last wave is fullest (the larger one on a tie) replaces the
    // rule above where it fills the waves at least a tenth better and its splits stay long (200 pages): short
    // splits are bound by their own latency, not by the waves (32K, one sequence: 43 us with 64 splits, 47 with 37).
    n_splits = min(n_splits, CKV_MAX_SPLITS);
    auto fill = [&](int n) { const long long ctas = (long long)units * n; return (double)ctas / (double)((ctas + sms - 1) / sms * sms); };
    const int lo = max(1, (3 * sms + 2 * units - 1) / (2 * units)), hi = min(max(lo, 42 * sms / (10 * units)), CKV_MAX_SPLITS);
    int best = lo;
    for (int n = lo; n <= hi; ++n)
      if (fill(n) >= fill(best)) best = n;
    if (fill(best) >= 1.1 * fill(n_splits) && total / best >= 200) n_splits = best;
  }
  if (mma && !dense) {
    // Up to 8 splits of a unit run as one cluster and merge in shared memory.  With so few units that 8 splits each
    // would leave most SMs idle, many short splits (merged through global memory) finish sooner.
    // (measured: about 1.75 CTAs per SM is the best grid there; more, shorter splits cost more in the merge)
    // Two of these CTAs fit an SM (shared memory): more than 2 * sms CTAs would run as two waves, the second one
    // waiting for the first (128 units: 3 splits each took 43 us, 2 splits each 34 us).
    const int by_sm = max(1, 2 * sms / units);
    n_splits = (by_sm > 8 && units * 16 <= sms) ? (7 * sms / 4 + units - 1) / units : min(by_sm, 8);
  }
  // at least one page per warp of a split: 8-warp CTAs everywhere except the tensor-core kernel's sparse mode (4 warps)
  const int min_pages = (mma && !dense) ? 4 : 8;
  n_splits = max(1, min(n_splits, min(CKV_MAX_SPLITS, (total + min_pages - 1) / min_pages)));
  int pps = (total + n_splits - 1) / n_splits;
  if (!(mma && !dense)) pps = (pps + 7) / 8 * 8;   // the tensor-core kernel deals pages to its warps one by one
  n_splits = max(1, (total + pps - 1) / pps);
  *n_splits_out = n_splits;
  *merged_out = mma && P.unit_done != nullptr;
  dim3 grid(n_splits, units);
  c->launches++;
  if (c->layout.kv_dtype == CKV_BF16)   // bf16 pages go through the tensor-core kernel
    return ckv_launch_attn_mma(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps,
                               scan_grid, out, lse, st);
  switch (P.G) {
    case 1: return launch_g<1>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 2: return launch_g<2>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 4: return launch_g<4>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 8: return launch_g<8>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t ckv_launch_merge(ckv_ctx *c, bool dense, const int *seq_lens, const int *sel_cnt, int n_splits,
                             int scan_grid, int batch, void *out, float *lse, cudaStream_t st) {
  const CkvDev &P = c->dev;
  dim3 grid(P.Hq, batch);
  const int units = batch * P.Hkv;
  if (c->layout.kv_dtype == CKV_BF16)
    ckv_merge_kernel<__nv_bfloat16><<<grid, CKV_D * kMergeGroups, 0, st>>>(P, seq_lens, sel_cnt, n_splits, scan_grid, units, dense,
                                                           (__nv_bfloat16 *)out, lse);
  else
    ckv_merge_kernel<float><<<grid, CKV_D * kMergeGroups, 0, st>>>(P, seq_lens, sel_cnt, n_splits, scan_grid, units, dense,
                                                    (float *)out, lse);
  c->launches++;
  return cudaGetLastError();
}
