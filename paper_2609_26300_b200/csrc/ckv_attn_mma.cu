// Exact attention over a list of cache pages on tensor cores (bf16 layout), split along the list, plus the
// removal of the selected blocks' mean-compensation terms (Eq. 12).  Same contract as the fp32-capable
// kernel in ckv_attn.cu: one partial (m, l, acc[128]) per (unit, split, head) for the merge kernel.
//
// Sparse mode: the page list of a unit is the pages of its selected blocks, in position order.
// Dense mode: every page of the sequence (Eq. 12 with S = all blocks; Sec. 3.1).
//
// A CTA takes a contiguous slice of the list; each of its 8 warps takes every 8th page.  A warp copies its
// page (16 tokens: a 4 KB K tile and a 4 KB V tile, each contiguous in the paged pool) into shared memory
// with 16-byte cp.async pieces whose destinations are XOR-swizzled by the token row, so that the matrix
// loads below are conflict-free; rows past the sequence end are zero-filled.  Then, with the G heads as the
// M dimension (rows 0..7 of 16) of mma.sync.m16n8k16:
//   S^T = Q K^T      heads x 16 tokens, Q fragments held in registers for the whole kernel
//   P   = 2^(S^T - m) per warp, running maximum raised only when exceeded by a slack; split into bf16 hi + lo
//   O  += P V        heads x 128 coordinates; the accumulator layout of S^T is the A-operand layout of P V
// For every selected block the scan kernel has already added the block's mean term |b| e^{zbar} vbar_b to
// the all-block compensation sum; here the same term is subtracted with one more P V-shaped product whose
// only non-zero row is the block's mean value (read as its stored hi + lo halves), so that
//   merge = exact(S) + mean(all) - mean(S) = exact(S) + mean(not S).
#include "ckv_internal.cuh"
#include "ckv_mma.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kTileBytes = CKV_PAGE * CKV_D * 2;      // one head's K (or V) page in bf16: 4 KB
constexpr int kRowBytes = CKV_D * 2;                  // 256
constexpr int kAuxBytes = 1536;                       // per warp: a mean-value row (512 B) per page buffer and a row of zeros
constexpr int kZeroRow = 1024;                        // offset of the row of zeros inside the aux area

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  // valid == false copies nothing and zero-fills the 16 bytes
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int G, bool DENSE>
__global__ void __launch_bounds__(kWarps * 32, DENSE ? 1 : 2)
ckv_attn_mma_kernel(CkvDev P, const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_pool,
                    const __nv_bfloat16 *__restrict__ v_pool, const int *__restrict__ page_table,
                    const int *__restrict__ seq_lens, const int *__restrict__ sel_ids,
                    const int *__restrict__ sel_cnt, int kcap, int pages_per_split, int nbuf) {
  extern __shared__ __align__(128) unsigned char smem[];   // [8 warps][nbuf][K tile | V tile], then [8 warps][aux]
  __shared__ __align__(16) float red[kWarps][G][CKV_PART_STRIDE];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int head = lane >> 2, qd = lane & 3;
  const bool hv = head < G;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int N = max(min(seq_lens[s], P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) / P.bs;
  const int nsel = DENSE ? X : min(sel_cnt[unit], kcap);
  const int total = DENSE ? (N + CKV_PAGE - 1) / CKV_PAGE : nsel * P.ppb;
  const bool comp = !DENSE && nsel < X;
  const int p0 = blockIdx.x * pages_per_split;
  const int p1 = min(p0 + pages_per_split, total);
  float *part = P.attn_part + ((size_t)unit * CKV_MAX_SPLITS + blockIdx.x) * G * CKV_PART_STRIDE;
  if (p0 >= total) {
    if (tid < G) { part[tid * CKV_PART_STRIDE] = -CUDART_INF_F; part[tid * CKV_PART_STRIDE + 1] = 0.f; }
    return;
  }

  unsigned char *wtiles = smem + (size_t)warp * nbuf * 2 * kTileBytes;
  unsigned char *waux = smem + (size_t)kWarps * nbuf * 2 * kTileBytes + (size_t)warp * kAuxBytes;
  const uint32_t aux_u32 = (uint32_t)__cvta_generic_to_shared(waux);
  // the row of zeros every unused row of the mean-value product points at
  if (lane < 16) reinterpret_cast<uint4 *>(waux + kZeroRow)[lane] = make_uint4(0u, 0u, 0u, 0u);

  // Q fragments: A operand rows 0..7 = heads, scaled logits come out of the products in log2 units
  uint32_t qa[8][2];
  {
    const __nv_bfloat16 *qrow = q + ((size_t)s * P.Hq + h * G + (hv ? head : 0)) * CKV_D;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const uint32_t v = __ldg(reinterpret_cast<const uint32_t *>(qrow + 16 * ks + 8 * hh + 2 * qd));
        qa[ks][hh] = hv ? v : 0u;
      }
  }
  const float sl2 = P.scale * kLog2e;

  float acc[16][2];
#pragma unroll
  for (int t = 0; t < 16; ++t) { acc[t][0] = 0.f; acc[t][1] = 0.f; }
  float m_ref = -CUDART_INF_F, l_acc = 0.f;
  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
  const int pshift = P.ppb == 1 ? 0 : (P.ppb == 2 ? 1 : 2);
  const int n_mine = (p1 - p0 - warp + kWarps - 1) / kWarps;   // this warp's pages: list index p0 + warp + 8 n
  const float2 *ls = P.ls + (size_t)unit * P.max_blocks * G;
  const __nv_bfloat16 *vmean = P.vmean + (size_t)unit * P.max_blocks * CKV_ROW_ELEMS;
  bool bad = false;

  struct PageRef { int phys, ntok, blk; bool first; };
  auto resolve = [&](int n) {
    PageRef r{-1, 0, -1, false};
    const int i = p0 + warp + kWarps * n;
    int page = i;
    bool ok = true;
    if (!DENSE) {
      r.blk = sel_ids[(size_t)unit * kcap + (i >> pshift)];
      ok = r.blk >= 0 && r.blk < X;
      if (!ok) r.blk = -1;
      page = (r.blk << pshift) + (i & (P.ppb - 1));
      r.first = ok && (i & (P.ppb - 1)) == 0;
    }
    if (ok) {
      r.ntok = min(CKV_PAGE, N - page * CKV_PAGE);
      if (r.ntok > 0) {
        r.phys = pt_row[page];
        if (r.phys < 0 || r.phys >= P.num_pages) { r.phys = -1; bad = true; }
      } else {
        r.ntok = 0;
      }
    }
    return r;
  };
  // start the copies of one page into buffer `buf`: 256 16-byte pieces per tile, 8 per lane; piece c of row r
  // lands at chunk c ^ (r & 7) of the row
  auto issue = [&](const PageRef &r, int buf) {
    if (r.phys >= 0) {
      const size_t src = ((size_t)r.phys * P.Hkv + h) * (CKV_PAGE * CKV_D);
      const uint32_t kb = (uint32_t)__cvta_generic_to_shared(wtiles + (size_t)buf * 2 * kTileBytes);
      const uint32_t vb = kb + kTileBytes;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int idx = lane + 32 * k, row = idx >> 4, c = idx & 15;
        const uint32_t off = (uint32_t)(row * kRowBytes + ((c ^ (row & 7)) << 4));
        const bool valid = row < r.ntok;
        const size_t so = src + (size_t)(valid ? row : 0) * CKV_D + 8 * c;
        cp_async16(kb + off, k_pool + so, valid);
        cp_async16(vb + off, v_pool + so, valid);
      }
      if (comp && r.first)   // the block's mean-value row, verbatim (hi halves then lo halves, swizzled by block index)
        cp_async16(aux_u32 + 512 * buf + 16 * lane, vmean + (size_t)r.blk * CKV_ROW_ELEMS + 8 * lane, true);
    }
    cp_async_commit();
  };

  PageRef cur = n_mine > 0 ? resolve(0) : PageRef{-1, 0, -1, false};
  if (n_mine > 0) issue(cur, 0);
  for (int n = 0, buf = 0; n < n_mine; ++n) {
    PageRef nxt{-1, 0, -1, false};
    const bool prefetch = nbuf > 1 && n + 1 < n_mine;
    if (prefetch) {
      nxt = resolve(n + 1);
      issue(nxt, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncwarp();
    if (cur.phys >= 0) {
      const uint32_t kb = (uint32_t)__cvta_generic_to_shared(wtiles + (size_t)buf * 2 * kTileBytes);
      const uint32_t vb = kb + kTileBytes;
      // ---- S^T = Q K^T: heads x 16 tokens (two n-tiles of 8 tokens) ----
      float sv[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, sv2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
      {
        const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int r = nt * 8 + lrow;
          const uint32_t rowaddr = kb + r * kRowBytes;
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // two 16-coordinate steps per ldmatrix.x4
            uint32_t b[4];
            ldmatrix_x4(b, rowaddr + (uint32_t)(((4 * j + lmat) ^ (r & 7)) << 4));
            mma_rows8(sv[nt][0], sv[nt][1], qa[2 * j][0], qa[2 * j][1], b[0], b[1]);
            mma_rows8(sv2[nt][0], sv2[nt][1], qa[2 * j + 1][0], qa[2 * j + 1][1], b[2], b[3]);
          }
          sv[nt][0] += sv2[nt][0]; sv[nt][1] += sv2[nt][1];
        }
      }
      // ---- softmax weights for this thread's head and its four tokens ----
      float tmax = -CUDART_INF_F;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool ok = hv && nt * 8 + 2 * qd + e < cur.ntok;
          sv[nt][e] = ok ? sv[nt][e] * sl2 : -CUDART_INF_F;
          tmax = fmaxf(tmax, sv[nt][e]);
        }
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
      if (tmax > m_ref + CKV_RESCALE_SLACK) {
        const float sc = exp2_diff(m_ref, tmax);
        m_ref = tmax;
        l_acc *= sc;
#pragma unroll
        for (int t = 0; t < 16; ++t) { acc[t][0] *= sc; acc[t][1] *= sc; }
      }
      uint32_t ph[2], pl[2];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float p[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          p[e] = sv[nt][e] == -CUDART_INF_F ? 0.f : fast_exp2(sv[nt][e] - m_ref);
          l_acc += p[e];
        }
        ph[nt] = pack_bf16(p[0], p[1]);
        pl[nt] = pack_bf16(p[0] - bf16_round(p[0]), p[1] - bf16_round(p[1]));
      }
      // ---- O += P V ----
      {
        const int r = ((lane >> 3) & 1) * 8 + (lane & 7);
        const uint32_t rowaddr = vb + r * kRowBytes;
        const int cpar = lane >> 4;
#pragma unroll
        for (int t2 = 0; t2 < 8; ++t2) {   // two 8-coordinate n-tiles per ldmatrix.x4
          uint32_t v[4];
          ldmatrix_x4_trans(v, rowaddr + (uint32_t)(((2 * t2 + cpar) ^ (r & 7)) << 4));
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], ph[0], ph[1], v[0], v[1]);
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], pl[0], pl[1], v[0], v[1]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], ph[0], ph[1], v[2], v[3]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], pl[0], pl[1], v[2], v[3]);
        }
      }
      if (comp && cur.first) {
        // take this block's mean term |b| e^{zbar} vbar_b back out (it is part of the all-block sum)
        float zl2 = -CUDART_INF_F;
        if (hv) {
          const float2 v = __ldg(ls + (size_t)head * P.max_blocks + cur.blk);
          zl2 = (v.x - 0.5f * v.y) * kLog2e;
        }
        if (zl2 > m_ref + CKV_RESCALE_SLACK) {
          const float sc = exp2_diff(m_ref, zl2);
          m_ref = zl2;
          l_acc *= sc;
#pragma unroll
          for (int t = 0; t < 16; ++t) { acc[t][0] *= sc; acc[t][1] *= sc; }
        }
        const float wbar = hv ? fast_exp2(zl2 - m_ref) : 0.f;
        if (qd == 0) l_acc -= wbar;
        // A operand: column 0 (the only real row of the B operand) holds -wbar for this thread's head
        const uint32_t wh = qd == 0 ? pack_bf16(-wbar, 0.f) : 0u;
        const uint32_t wl = qd == 0 ? pack_bf16(-(wbar - bf16_round(wbar)), 0.f) : 0u;
        // B operand rows: row 0 is the mean-value row, every other row the row of zeros
        const bool row0 = (lane & 15) == 0;   // lanes 0 and 16 address row 0 of their 8x8 matrices (chunks c, c + 1)
        const int cpar = lane >> 4;
#pragma unroll
        for (int t2 = 0; t2 < 8; ++t2) {
          const uint32_t coff = (uint32_t)(swz_chunk(2 * t2 + cpar, cur.blk) << 4);
          uint32_t vh[4], vl[4];
          ldmatrix_x4_trans(vh, row0 ? aux_u32 + 512 * buf + coff : aux_u32 + kZeroRow);
          ldmatrix_x4_trans(vl, row0 ? aux_u32 + 512 * buf + 256 + coff : aux_u32 + kZeroRow);
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh, 0u, vh[0], vh[1]);
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wl, 0u, vh[0], vh[1]);
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh, 0u, vl[0], vl[1]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh, 0u, vh[2], vh[3]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wl, 0u, vh[2], vh[3]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh, 0u, vl[2], vl[3]);
        }
      }
    }
    __syncwarp();   // the buffer (and the mean-value row) may be overwritten from here on
    if (nbuf > 1) {
      cur = nxt;
      buf ^= 1;
    } else if (n + 1 < n_mine) {
      cur = resolve(n + 1);
      issue(cur, 0);
    }
  }
  cp_async_wait<0>();
  if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);

  // ---- CTA partial: fold the warps (each with its own running maximum) ----
  l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 1);
  l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 2);
  if (hv) {
    float *r = red[warp][head];
#pragma unroll
    for (int t = 0; t < 16; ++t) *reinterpret_cast<float2 *>(r + 4 + 8 * t + 2 * qd) = make_float2(acc[t][0], acc[t][1]);
    if (qd == 0) { r[0] = m_ref; r[1] = l_acc; }
  }
  __syncthreads();
  for (int idx = tid; idx < G * CKV_D; idx += kWarps * 32) {
    const int g = idx / CKV_D, c = idx % CKV_D;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, red[w][g][0]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float sc = exp2_diff(red[w][g][0], M);
      num = fmaf(red[w][g][4 + c], sc, num);
      den = fmaf(red[w][g][1], sc, den);
    }
    part[g * CKV_PART_STRIDE + 4 + c] = num;
    if (c == 0) { part[g * CKV_PART_STRIDE] = M; part[g * CKV_PART_STRIDE + 1] = den; }
  }
}

inline size_t static_smem(int G) { return (size_t)kWarps * G * CKV_PART_STRIDE * 4 + 256; }
inline size_t dyn_smem(int nbuf) { return (size_t)kWarps * (nbuf * 2 * kTileBytes + kAuxBytes); }

template <int G>
cudaError_t launch_g(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                     const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt, int kcap,
                     dim3 grid, int pps, cudaStream_t st) {
  const int nbuf = (dense || pps > kWarps) ? 2 : 1;
  const size_t smem = dyn_smem(nbuf);
  const __nv_bfloat16 *qp = (const __nv_bfloat16 *)q, *kp = (const __nv_bfloat16 *)k_pool, *vp = (const __nv_bfloat16 *)v_pool;
  if (dense)
    ckv_attn_mma_kernel<G, true><<<grid, kWarps * 32, smem, st>>>(c->dev, qp, kp, vp, page_table, seq_lens, sel_ids,
                                                                  sel_cnt, kcap, pps, nbuf);
  else
    ckv_attn_mma_kernel<G, false><<<grid, kWarps * 32, smem, st>>>(c->dev, qp, kp, vp, page_table, seq_lens, sel_ids,
                                                                   sel_cnt, kcap, pps, nbuf);
  return cudaGetLastError();
}

template <int G>
cudaError_t configure_g() {
  const int smem = (int)dyn_smem(2);
  cudaError_t e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return e;
}

}  // namespace

cudaError_t ckv_configure_attn_mma(const ckv_ctx *c) {
  switch (c->dev.G) {
    case 1: return configure_g<1>();
    case 2: return configure_g<2>();
    case 4: return configure_g<4>();
    case 8: return configure_g<8>();
  }
  return cudaErrorInvalidValue;
}

cudaError_t ckv_launch_attn_mma(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                                const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt,
                                int kcap, dim3 grid, int pps, cudaStream_t st) {
  switch (c->dev.G) {
    case 1: return launch_g<1>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 2: return launch_g<2>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 4: return launch_g<4>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
    case 8: return launch_g<8>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, st);
  }
  return cudaErrorInvalidValue;
}
