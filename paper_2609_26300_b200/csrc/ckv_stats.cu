// Block summaries: prefill-time build and per-token append (Sec. 4.1-4.2, Eq. 8 right half).
//
// One warp owns one block.  A token row (128 elements) is spread over the 16 lanes of a half
// warp, 8 consecutive coordinates per lane (one 16-byte load for bf16); the two half warps take
// alternate rows.  Means and squared deviations are accumulated in fp32 in two passes (mean
// first, then deviations from it) over a page of rows held in registers; the pages of a longer
// block are joined pairwise (ckv_blockstats.cuh).  Build, append and chunked prefill run the same
// operations in the same order, so their results are bit-identical.
#include "ckv_internal.cuh"
#include "ckv_blockstats.cuh"

namespace {

constexpr int kBuildRounds = 8;   // blocks per warp of the build kernel
constexpr int kPrefillRounds = 4; // blocks per warp of the prefill kernel's register-resident variant

// A warp takes kBuildRounds blocks, eight blocks apart.  Two CTAs per SM: the block routine holds a page's 16 key and
// 16 value rows in registers, which does not fit three CTAs' register share without spills, and the kernel was bound
// by instruction issue, not by DRAM, while it spilled.  The 16 warps of an SM keep enough rows in flight by
// themselves: asking the L2 for a warp's next block ahead of time (which paid while the block routine was long) now
// only costs instructions, and with blocks of several pages it cost a third of the time.
// ONEP: one-page blocks of bf16 rows (the default layout), compiled without the other paths of the block routine.
template <typename T, bool ONEP>
__global__ void __launch_bounds__(256, 2) ckv_stats_build_kernel(CkvDev P, const T *__restrict__ k_pool,
                                                              const T *__restrict__ v_pool,
                                                              const int *__restrict__ page_table,
                                                              const int *__restrict__ seq_lens) {
  __shared__ float sq_smem[8][CKV_D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int N = min(seq_lens[s], P.max_blocks * P.bs);
  const int X = (N + P.bs - 1) / P.bs;
  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
#pragma unroll 1
  for (int i = 0; i < kBuildRounds; ++i) {
    const int b = (blockIdx.x * kBuildRounds + i) * 8 + warp;
    if (b >= X) return;
    const int cnt = min(P.bs, N - b * P.bs);
    const size_t row = (size_t)unit * P.max_blocks + b;
    block_stats_warp<T, true, ONEP>(P, k_pool, v_pool, pt_row, h, b, cnt, sq_smem[warp], P.kmean + row * P.row_elems,
                                    P.dbar + row * P.r, P.vmean + row * P.row_elems, lane);
  }
}

// One CTA per sequence, one warp per KV head (looping when there are more heads than warps).
template <typename T>
__global__ void __launch_bounds__(256) ckv_append_kernel(CkvDev P, T *k_pool, T *v_pool,
                                                         const int *__restrict__ page_table, int *seq_lens,
                                                         const T *__restrict__ k_new, const T *__restrict__ v_new) {
  __shared__ float sq_smem[8][CKV_D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int s = blockIdx.x;
  const int N = seq_lens[s];
  // the new row of this warp's first head does not depend on N: it is requested together with it, so that the
  // chain length -> page -> row has no fourth link (16-byte pieces: lanes 0-15 hold K, lanes 16-31 hold V)
  constexpr int PIECES = (int)(CKV_D * sizeof(T) / 16);
  constexpr int PP = PIECES / 16;
  uint4 fresh[PP];
  if (warp < P.Hkv) {
    const uint4 *src = reinterpret_cast<const uint4 *>((lane < 16 ? k_new : v_new) + ((size_t)s * P.Hkv + warp) * CKV_D);
#pragma unroll
    for (int k = 0; k < PP; ++k) fresh[k] = __ldg(src + (lane & 15) + 16 * k);
  }
  __syncthreads();   // every warp has read N before thread 0 may change it
  if (N < 0 || N >= P.max_blocks * P.bs) {
    if (threadIdx.x == 0) atomicOr(P.status, CKV_DEV_SEQ_FULL);
    return;
  }
  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
  const int page = N / CKV_PAGE, slot = N % CKV_PAGE;
  const int phys = pt_row[page];
  const bool ok = phys >= 0 && phys < P.num_pages;
  const int b = N / P.bs, cnt = N + 1 - b * P.bs;
  for (int h = warp; h < P.Hkv; h += nwarps) {
    if (ok) {
      if (h != warp) {   // further heads of this warp (more KV heads than warps)
        const uint4 *src = reinterpret_cast<const uint4 *>((lane < 16 ? k_new : v_new) + ((size_t)s * P.Hkv + h) * CKV_D);
#pragma unroll
        for (int k = 0; k < PP; ++k) fresh[k] = __ldg(src + (lane & 15) + 16 * k);
      }
      uint4 *dst = reinterpret_cast<uint4 *>((lane < 16 ? k_pool : v_pool) +
                                             (((size_t)phys * P.Hkv + h) * CKV_PAGE + slot) * CKV_D);
#pragma unroll
      for (int k = 0; k < PP; ++k) dst[(lane & 15) + 16 * k] = fresh[k];
    }
    __syncwarp();
    const size_t row = ((size_t)s * P.Hkv + h) * P.max_blocks + b;
    block_stats_warp<T, false>(P, k_pool, v_pool, pt_row, h, b, cnt, sq_smem[warp], P.kmean + row * P.row_elems,
                               P.dbar + row * P.r, P.vmean + row * P.row_elems, lane);
  }
  __syncthreads();
  if (threadIdx.x == 0) seq_lens[s] = N + 1;
}

// Chunked prefill: new_lens[s] tokens per sequence arrive as contiguous rows; one warp per touched block copies the
// block's new rows into their pages and then runs the block routine over the block (rows that were already in the
// cache included), so the new keys and values cross DRAM once on the way in and the summaries come out of the same
// pass.  The CTA that finishes last stores the new sequence lengths (every warp read the old ones when it started).
// REG: 1 = one-page blocks of bf16 rows (the default layout), 2 = bf16 blocks of several pages: the variants whose
// rows never leave the registers; 0 = the general form (fp32 pages).
template <typename T, int REG>
__global__ void __launch_bounds__(256, REG ? 2 : 1) ckv_prefill_kernel(CkvDev P, T *k_pool, T *v_pool,
                                                          const int *__restrict__ page_table, int *seq_lens,
                                                          const T *__restrict__ k_src, const T *__restrict__ v_src,
                                                          const int *__restrict__ new_lens, int src_stride, int batch) {
  __shared__ float sq_smem[8][CKV_D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int cap = P.max_blocks * P.bs;
  const int N = seq_lens[s], M = new_lens[s];
  const int m_eff = N < 0 ? 0 : max(min(min(M, src_stride), cap - N), 0);   // tokens that fit
  if (M > m_eff && blockIdx.x == 0 && threadIdx.x == 0) atomicOr(P.status, CKV_DEV_SEQ_FULL);
  // the register-resident variant gives a warp kPrefillRounds blocks, eight blocks apart (L2 requests for the next
  // block's rows ahead of time made it slower once the block routine had been trimmed: 763 against 728 us)
  constexpr int kRounds = REG ? kPrefillRounds : 1;
#pragma unroll 1
  for (int rnd = 0; rnd < kRounds; ++rnd) {
  const int b = (N >= 0 ? N / P.bs : 0) + (blockIdx.x * kRounds + rnd) * 8 + warp;
  if (m_eff > 0 && b <= (N + m_eff - 1) / P.bs) {
    const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
    const int p_lo = max(b * P.bs, N), p_hi = min((b + 1) * P.bs, N + m_eff);
    if constexpr (REG != 0) {
      // bf16 rows: the rows of a page go from the chunk into registers in the layout the block routine works in (rows
      // of the block that were already in the cache come from the page), the new ones are stored to the page, and the
      // summaries are worked out from the registers -- the chunk crosses DRAM once and nothing is read back.  A block of
      // several pages is joined page by page, exactly as the block routine does it (same bits).
      const int hw = lane >> 4, li = lane & 15;
      const int cnt = min(P.bs, N + m_eff - b * P.bs);
      bool bad = false;
      // page pg of the block: its mean key, value sums and this half warp's squared deviations; false: bad page id
      auto page = [&](int pg, int ntok, float (&mb)[8], float (&vb)[8], float (&qb)[8]) -> bool {
        const int phys = pt_row[b * P.ppb + pg];
        if (phys < 0 || phys >= P.num_pages) return false;
        const size_t pbase = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
        const int pfirst = b * P.bs + pg * CKV_PAGE;   // position of the page's first row
        uint4 kraw[8], vraw[8];
        if (ntok == CKV_PAGE && pfirst >= N) {
          // a full page made of new rows only (all but the first and last touched page): no per-row tests
          const size_t so = (((size_t)s * src_stride + (pfirst + hw - N)) * P.Hkv + h) * CKV_D + 8 * li;
          const size_t sstep = (size_t)2 * P.Hkv * CKV_D;   // two chunk rows on
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            kraw[j] = __ldg(reinterpret_cast<const uint4 *>(k_src + so + j * sstep));
            vraw[j] = __ldg(reinterpret_cast<const uint4 *>(v_src + so + j * sstep));
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            *reinterpret_cast<uint4 *>(k_pool + pbase + (size_t)(hw + 2 * j) * CKV_D) = kraw[j];
            *reinterpret_cast<uint4 *>(v_pool + pbase + (size_t)(hw + 2 * j) * CKV_D) = vraw[j];
          }
          block_stats_rows16<true>(kraw, vraw, true, CKV_PAGE, lane, mb, vb, qb);
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int t = hw + 2 * j, p = pfirst + t;
            const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
            kraw[j] = zero; vraw[j] = zero;
            if (t < ntok) {
              if (p >= p_lo) {
                const size_t so = (((size_t)s * src_stride + (p - N)) * P.Hkv + h) * CKV_D + 8 * li;
                kraw[j] = __ldg(reinterpret_cast<const uint4 *>(k_src + so));
                vraw[j] = __ldg(reinterpret_cast<const uint4 *>(v_src + so));
              } else {
                kraw[j] = *reinterpret_cast<const uint4 *>(k_pool + pbase + (size_t)t * CKV_D);
                vraw[j] = *reinterpret_cast<const uint4 *>(v_pool + pbase + (size_t)t * CKV_D);
              }
            }
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int t = hw + 2 * j, p = pfirst + t;
            if (t < ntok && p >= p_lo) {
              *reinterpret_cast<uint4 *>(k_pool + pbase + (size_t)t * CKV_D) = kraw[j];
              *reinterpret_cast<uint4 *>(v_pool + pbase + (size_t)t * CKV_D) = vraw[j];
            }
          }
          block_stats_rows16(kraw, vraw, true, ntok, lane, mb, vb, qb);
        }
        return true;
      };
      float km[8], vs[8], sq[8];
      if constexpr (REG == 1) {   // one-page blocks (the default layout)
        if (!page(0, cnt, km, vs, sq)) {
          bad = true;
#pragma unroll
          for (int i = 0; i < 8; ++i) { km[i] = 0.f; vs[i] = 0.f; sq[i] = 0.f; }
        }
      } else {
        float na = 0.f, m2[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { km[i] = 0.f; vs[i] = 0.f; m2[i] = 0.f; }
        const int npages = (cnt + CKV_PAGE - 1) / CKV_PAGE;
#pragma unroll 1
        for (int pg = 0; pg < npages; ++pg) {
          const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
          float mb[8], vb[8], qb[8];
          if (!page(pg, ntok, mb, vb, qb)) { bad = true; continue; }
#pragma unroll
          for (int i = 0; i < 8; ++i) qb[i] += __shfl_xor_sync(0xffffffffu, qb[i], 16);
          combine_pages(na, km, m2, vs, ntok, mb, qb, vb);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sq[i] = hw == 0 ? m2[i] : 0.f;
      }
      const size_t row = (size_t)unit * P.max_blocks + b;
      block_stats_finish(P, b, (float)cnt, km, vs, sq, sq_smem[warp], P.kmean + row * P.row_elems, P.dbar + row * P.r,
                         P.vmean + row * P.row_elems, lane, bad);
    }
    if constexpr (REG == 0) {
    constexpr int PIECES = (int)(CKV_D * sizeof(T) / 16);   // 16-byte pieces of a row: 16 (bf16) or 32 (fp32)
    constexpr int PP = PIECES / 16;                          // pieces per lane and row
    bool bad = false;
    const T *src_base = (lane < 16 ? k_src : v_src);         // lanes 0-15 copy K, lanes 16-31 copy V
    T *dst_base = (lane < 16 ? k_pool : v_pool);
    for (int pg = p_lo / CKV_PAGE; pg * CKV_PAGE < p_hi; ++pg) {
      const int phys = pt_row[pg];
      if (phys < 0 || phys >= P.num_pages) { bad = true; continue; }
      // all rows of the page are requested before any is stored
      uint4 r[CKV_PAGE][PP];
#pragma unroll
      for (int t = 0; t < CKV_PAGE; ++t) {
        const int p = pg * CKV_PAGE + t;
        if (p >= p_lo && p < p_hi) {
          const uint4 *src = reinterpret_cast<const uint4 *>(src_base + (((size_t)s * src_stride + (p - N)) * P.Hkv + h) * CKV_D);
#pragma unroll
          for (int k = 0; k < PP; ++k) r[t][k] = __ldg(src + (lane & 15) + 16 * k);
        }
      }
#pragma unroll
      for (int t = 0; t < CKV_PAGE; ++t) {
        const int p = pg * CKV_PAGE + t;
        if (p >= p_lo && p < p_hi) {
          uint4 *dst = reinterpret_cast<uint4 *>(dst_base + (((size_t)phys * P.Hkv + h) * CKV_PAGE + t) * CKV_D);
#pragma unroll
          for (int k = 0; k < PP; ++k) dst[(lane & 15) + 16 * k] = r[t][k];
        }
      }
    }
    if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);
    __syncwarp();
    const int cnt = min(P.bs, N + m_eff - b * P.bs);
    const size_t row = (size_t)unit * P.max_blocks + b;
    block_stats_warp<T, false>(P, k_pool, v_pool, pt_row, h, b, cnt, sq_smem[warp], P.kmean + row * P.row_elems,
                               P.dbar + row * P.r, P.vmean + row * P.row_elems, lane);
    }
  }
  }   // rounds
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(P.unit_done, 1) == (int)(gridDim.x * gridDim.y) - 1) {
      P.unit_done[0] = 0;
      for (int i = 0; i < batch; ++i) {
        const int n = seq_lens[i];
        if (n >= 0) seq_lens[i] = n + max(min(min(new_lens[i], src_stride), cap - n), 0);
      }
    }
  }
}

// Summaries as plain fp32 arrays (hi + lo, chunks back in coordinate order): one warp per block row.
__global__ void __launch_bounds__(256) ckv_stats_export_kernel(CkvDev P, int rows, float *__restrict__ kmean,
                                                               float *__restrict__ dbar, float *__restrict__ vmean) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int b = row % P.max_blocks, hw = lane >> 4, li = lane & 15;
  float x[8];
  load_split8((hw == 0 ? P.kmean : P.vmean) + (size_t)row * P.row_elems, li, b, x, P.row_elems == CKV_ROW_ELEMS);
  float *dst = (hw == 0 ? kmean : vmean) + (size_t)row * CKV_D + 8 * li;
  reinterpret_cast<float4 *>(dst)[0] = make_float4(x[0], x[1], x[2], x[3]);
  reinterpret_cast<float4 *>(dst)[1] = make_float4(x[4], x[5], x[6], x[7]);
  if (P.r == CKV_D) {
    if (hw == 0) {
      load_split8(reinterpret_cast<const __nv_bfloat16 *>(P.dbar + (size_t)row * CKV_D), li, b, x);
      float *dd = dbar + (size_t)row * CKV_D + 8 * li;
      reinterpret_cast<float4 *>(dd)[0] = make_float4(x[0], x[1], x[2], x[3]);
      reinterpret_cast<float4 *>(dd)[1] = make_float4(x[4], x[5], x[6], x[7]);
    }
  } else {
    for (int t = lane; t < P.r; t += 32) dbar[(size_t)row * P.r + t] = P.dbar[(size_t)row * P.r + t];
  }
}

}  // namespace

cudaError_t ckv_launch_stats_export(ckv_ctx *c, int batch, float *kmean, float *dbar, float *vmean, cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int rows = batch * P.Hkv * P.max_blocks;
  ckv_stats_export_kernel<<<(rows + 7) / 8, 256, 0, st>>>(P, rows, kmean, dbar, vmean);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ckv_launch_stats_build(ckv_ctx *c, const void *k_pool, const void *v_pool, const int *page_table,
                                   const int *seq_lens, int batch, int max_len, cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int xmax = (max_len + P.bs - 1) / P.bs;
  if (xmax <= 0 || batch <= 0) return cudaSuccess;
  dim3 grid((xmax + 8 * kBuildRounds - 1) / (8 * kBuildRounds), batch * P.Hkv);
  if (c->layout.kv_dtype == CKV_BF16 && P.ppb == 1)
    ckv_stats_build_kernel<__nv_bfloat16, true><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16 *)k_pool,
                                                                      (const __nv_bfloat16 *)v_pool, page_table, seq_lens);
  else if (c->layout.kv_dtype == CKV_BF16)
    ckv_stats_build_kernel<__nv_bfloat16, false><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16 *)k_pool,
                                                                       (const __nv_bfloat16 *)v_pool, page_table, seq_lens);
  else
    ckv_stats_build_kernel<float, false><<<grid, 256, 0, st>>>(P, (const float *)k_pool, (const float *)v_pool, page_table,
                                                               seq_lens);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ckv_launch_prefill(ckv_ctx *c, void *k_pool, void *v_pool, const int *page_table, int *seq_lens,
                               const void *k_src, const void *v_src, const int *new_lens, int src_stride, int batch,
                               int max_new, cudaStream_t st) {
  const CkvDev &P = c->dev;
  if (batch <= 0 || max_new <= 0) return cudaSuccess;
  const int touched = (max_new + P.bs - 1) / P.bs + 1;   // a chunk that starts inside a block touches one more
  dim3 grid((touched + 7) / 8, batch * P.Hkv);
  const dim3 grid_one((touched + 8 * kPrefillRounds - 1) / (8 * kPrefillRounds), batch * P.Hkv);
  if (c->layout.kv_dtype == CKV_BF16 && P.ppb == 1)
    ckv_prefill_kernel<__nv_bfloat16, 1><<<grid_one, 256, 0, st>>>(P, (__nv_bfloat16 *)k_pool, (__nv_bfloat16 *)v_pool,
                                                                  page_table, seq_lens, (const __nv_bfloat16 *)k_src,
                                                                  (const __nv_bfloat16 *)v_src, new_lens, src_stride, batch);
  else if (c->layout.kv_dtype == CKV_BF16)
    ckv_prefill_kernel<__nv_bfloat16, 2><<<grid_one, 256, 0, st>>>(P, (__nv_bfloat16 *)k_pool, (__nv_bfloat16 *)v_pool,
                                                                   page_table, seq_lens, (const __nv_bfloat16 *)k_src,
                                                                   (const __nv_bfloat16 *)v_src, new_lens, src_stride, batch);
  else
    ckv_prefill_kernel<float, 0><<<grid, 256, 0, st>>>(P, (float *)k_pool, (float *)v_pool, page_table, seq_lens,
                                                    (const float *)k_src, (const float *)v_src, new_lens, src_stride, batch);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ckv_launch_append(ckv_ctx *c, void *k_pool, void *v_pool, const int *page_table, int *seq_lens,
                              const void *k_new, const void *v_new, int batch, cudaStream_t st) {
  const CkvDev &P = c->dev;
  if (batch <= 0) return cudaSuccess;
  const int threads = 32 * min(P.Hkv, 8);
  if (c->layout.kv_dtype == CKV_BF16)
    ckv_append_kernel<__nv_bfloat16><<<batch, threads, 0, st>>>(P, (__nv_bfloat16 *)k_pool, (__nv_bfloat16 *)v_pool,
                                                                page_table, seq_lens, (const __nv_bfloat16 *)k_new,
                                                                (const __nv_bfloat16 *)v_new);
  else
    ckv_append_kernel<float><<<batch, threads, 0, st>>>(P, (float *)k_pool, (float *)v_pool, page_table, seq_lens,
                                                        (const float *)k_new, (const float *)v_new);
  c->launches++;
  return cudaGetLastError();
}
