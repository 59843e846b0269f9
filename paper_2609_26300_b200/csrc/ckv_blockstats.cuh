// The block-summary routine shared by the prefill-time build, the per-token append and the chunked prefill
// (Sec. 4.1-4.2, Eq. 8 right half): one warp works out mean key, grouped variance and mean value of one block.
//
// A token row (128 elements) is spread over the 16 lanes of a half warp, 8 consecutive coordinates per lane (one
// 16-byte load for bf16); the two half warps take alternate rows.  Means and squared deviations are accumulated in
// fp32 in two passes (mean first, then deviations from it) over the rows of a page held in registers or shared
// memory; a block of several bf16 pages is read once, page after page, and the pages' (count, mean, squared
// deviations) are combined with the pairwise update of Chan et al. (combine_pages).  Every caller runs the same
// operations in the same order, so a block's summary has the same bits whichever way it was produced.
#ifndef CKV_BLOCKSTATS_CUH_
#define CKV_BLOCKSTATS_CUH_
#include "ckv_internal.cuh"

// Second half of the block routine, shared by its variants: the half warps' squared deviations are combined, the
// three summary rows are written (hw 0: mean key and variances, hw 1: mean value).  km: mean key, vs: value sums,
// sq: this half warp's squared deviations, all for the lane's 8 coordinates.
__device__ __forceinline__ void block_stats_finish(const CkvDev &P, int b, float fc, const float (&km)[8],
                                                   const float (&vs)[8], float (&sq)[8], float *sq_smem,
                                                   __nv_bfloat16 *kmean_row, float *dbar_row,
                                                   __nv_bfloat16 *vmean_row, int lane, bool bad) {
  const int hw = lane >> 4, li = lane & 15;
  const float inv = 1.0f / fc;
#pragma unroll
  for (int i = 0; i < 8; ++i) sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], 16);
  // the two mean rows leave through one store routine: half warp 0 writes the mean key, half warp 1 the mean value
  {
    float rowv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) rowv[i] = hw == 0 ? km[i] : vs[i] * inv;
    store_split8(hw == 0 ? kmean_row : vmean_row, li, b, rowv, P.row_elems == CKV_ROW_ELEMS);
  }
  const int gs = CKV_D / P.r;
  const int run = P.glayout == 0 ? gs : gs / 2;   // consecutive coordinates of a group (two runs, 64 apart, in layout 1)
  if (P.r == CKV_D) {
    // one group per coordinate: the variance row has the mean rows' layout (split bf16 pairs, swizzled chunks),
    // so that the scan can project it with the same tensor-core product as the mean keys
    if (hw == 0) {
      float dv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) dv[i] = sq[i] * inv;
      store_split8(reinterpret_cast<__nv_bfloat16 *>(dbar_row), li, b, dv);
    }
  } else if (run >= 8) {
    // grouped variance: average of the per-coordinate population variances of each group (Eq. 8).  A run is a
    // whole number of lanes: the lane's eight coordinates first, then the lanes of the run, then the second run.
    float ps = ((sq[0] + sq[1]) + (sq[2] + sq[3])) + ((sq[4] + sq[5]) + (sq[6] + sq[7]));
    const int w = run >> 3;
    for (int o = 1; o < w; o <<= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    if (P.glayout != 0) ps += __shfl_xor_sync(0xffffffffu, ps, 8);
    const int lg = P.glayout == 0 ? li : (li & 7);
    if (hw == 0 && (lg & (w - 1)) == 0 && (P.glayout == 0 || li < 8)) dbar_row[lg / w] = ps / (fc * (float)gs);
  } else {
    // groups narrower than a lane's eight coordinates: through shared memory
    if (hw == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) sq_smem[8 * li + i] = sq[i];
    }
    __syncwarp();
    for (int t = lane; t < P.r; t += 32) {
      float s = 0.f;
      if (P.glayout == 0) {
        for (int i = 0; i < gs; ++i) s += sq_smem[t * gs + i];
      } else {
        const int hg = gs / 2;
        for (int i = 0; i < hg; ++i) s += sq_smem[t * hg + i];
        for (int i = 0; i < hg; ++i) s += sq_smem[CKV_D / 2 + t * hg + i];
      }
      dbar_row[t] = s / (fc * (float)gs);
    }
    __syncwarp();
  }
  if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);
}

// Running (count, mean key, squared deviations from it, value sums) of the pages seen so far, joined with those of
// one more page of nb rows: delta = m_b - m_a, m = m_a + delta n_b / n, M2 = M2_a + M2_b + delta^2 n_a n_b / n.
// Everything is per coordinate and the same in all lanes that hold the coordinate; the first page only initialises.
__device__ __forceinline__ void combine_pages(float &na, float (&mean)[8], float (&m2)[8], float (&vsum)[8], int nb,
                                              const float (&mb)[8], const float (&m2b)[8], const float (&vb)[8]) {
  if (na == 0.f) {
#pragma unroll
    for (int i = 0; i < 8; ++i) { mean[i] = mb[i]; m2[i] = m2b[i]; vsum[i] = vb[i]; }
    na = (float)nb;
    return;
  }
  const float fb = (float)nb, n = na + fb;
  const float wb = fb / n, wab = na * wb;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float d = mb[i] - mean[i];
    mean[i] = fmaf(d, wb, mean[i]);
    m2[i] = fmaf(d * d, wab, m2[i] + m2b[i]);
    vsum[i] += vb[i];
  }
  na = n;
}

// The two passes over a one-page block of bf16 rows held in registers: lane (hw, li) holds the 8 coordinates 8 li ..
// of the key and value rows hw, hw + 2, ... (rows that do not exist: zeros, and they are skipped).  Leaves the mean
// key (km), the value sums (vs) and this half warp's squared deviations (sq) for block_stats_finish.  Every caller
// that has such a block's rows in registers uses this one routine, so the summaries have the same bits whether the
// rows came from the pool or from a prefill chunk on its way into the pool.
// FULL: the caller knows that all 16 rows exist (ok, cnt == 16): the same operations without the per-row tests.
template <bool FULL = false>
__device__ __forceinline__ void block_stats_rows16(const uint4 (&kraw)[8], const uint4 (&vraw)[8], bool ok, int cnt,
                                                   int lane, float (&km)[8], float (&vs)[8], float (&sq)[8]) {
  const int hw = lane >> 4;
  const float inv = 1.0f / (float)cnt;   // the reciprocal every routine of this file divides by (exact for 16-token blocks)
  float ks[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { ks[i] = 0.f; vs[i] = 0.f; }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (FULL || (ok && hw + 2 * j < cnt)) {
      // mixed-precision adds: a bf16 operand widened inside the instruction (exact), the same sum as ks[i] += float(k)
      add_bf16x8(kraw[j], ks);
      add_bf16x8(vraw[j], vs);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    ks[i] += __shfl_xor_sync(0xffffffffu, ks[i], 16);
    vs[i] += __shfl_xor_sync(0xffffffffu, vs[i], 16);
    km[i] = ks[i] * inv;
    sq[i] = 0.f;
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (FULL || (ok && hw + 2 * j < cnt)) {
      float dv[8];
      sub_bf16x8(kraw[j], km, dv);   // float(k) - km
#pragma unroll
      for (int i = 0; i < 8; ++i) sq[i] = fmaf(dv[i], dv[i], sq[i]);
    }
  }
}

// NC: the pools are read-only for the whole kernel (loads may use the non-coherent path).
// ONEP: the caller's layout has one-page blocks of bf16 rows, and only that path is compiled (fewer registers).
// sq_smem: 128 floats of shared memory owned by the calling warp.
template <typename T, bool NC, bool ONEP = false>
__device__ __forceinline__ void block_stats_warp(const CkvDev &P, const T *__restrict__ k_pool,
                                                 const T *__restrict__ v_pool, const int *__restrict__ pt_row,
                                                 int h, int b, int cnt, float *sq_smem, __nv_bfloat16 *kmean_row,
                                                 float *dbar_row, __nv_bfloat16 *vmean_row, int lane) {
  const int hw = lane >> 4, li = lane & 15;
  float ks[8], vs[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { ks[i] = 0.f; vs[i] = 0.f; }
  const int npages = (cnt + CKV_PAGE - 1) / CKV_PAGE;
  bool bad = false;
  const float fc = (float)cnt, inv = 1.0f / fc;
  float km[8], sq[8];
  bool done = false;
  if constexpr (sizeof(T) == 2) {
    if (npages == 1) {
      // One page of bf16 rows (every block of the default 16-token layout): the key rows stay in registers between
      // the two passes, so the cache is read exactly once.
      done = true;
      const int phys = pt_row[b * P.ppb];
      const bool ok = phys >= 0 && phys < P.num_pages;
      bad = !ok;
      const size_t base = ok ? ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li : 0;
      uint4 kraw[8], vraw[8];
      const uint4 *kp = reinterpret_cast<const uint4 *>(k_pool + base + (size_t)hw * CKV_D);
      const uint4 *vp = reinterpret_cast<const uint4 *>(v_pool + base + (size_t)hw * CKV_D);
      constexpr int kStep = 2 * CKV_D / 8;   // two rows on, in 16-byte units
      if (ok && cnt == CKV_PAGE) {   // a full block (all but the last of a sequence): no per-row tests
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          kraw[j] = NC ? __ldg(kp + j * kStep) : kp[j * kStep];
          vraw[j] = NC ? __ldg(vp + j * kStep) : vp[j * kStep];
        }
        block_stats_rows16<true>(kraw, vraw, true, CKV_PAGE, lane, km, vs, sq);
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const bool valid = ok && hw + 2 * j < cnt;
          const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
          kraw[j] = valid ? (NC ? __ldg(kp + j * kStep) : kp[j * kStep]) : zero;
          vraw[j] = valid ? (NC ? __ldg(vp + j * kStep) : vp[j * kStep]) : zero;
        }
        block_stats_rows16(kraw, vraw, ok, cnt, lane, km, vs, sq);
      }
    }
  }
  if constexpr (sizeof(T) == 2 && !ONEP) {
    if (!done) {
      // Several pages of bf16 rows (32- and 64-token blocks): every page goes through the registers once -- its own
      // two passes, as for a one-page block -- and is joined to the pages before it.  When the caller works on one
      // block only (the append, the chunked prefill) the L2 is asked for all pages first, so that only the first one
      // costs a DRAM round trip.  (The build kernel asks for its next block itself.)
      done = true;
      if constexpr (!NC) {
        if (lane < npages) {
          const int phys = pt_row[b * P.ppb + lane];
          if (phys >= 0 && phys < P.num_pages) {
            const size_t off = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D;
            const unsigned bytes = CKV_PAGE * CKV_D * sizeof(T);
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(k_pool + off), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(v_pool + off), "r"(bytes) : "memory");
          }
        }
      }
      float na = 0.f, m2[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { km[i] = 0.f; m2[i] = 0.f; }
#pragma unroll 1
      for (int pg = 0; pg < npages; ++pg) {
        const int phys = pt_row[b * P.ppb + pg];
        if (phys < 0 || phys >= P.num_pages) { bad = true; continue; }
        const size_t base = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
        const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
        const uint4 *kp = reinterpret_cast<const uint4 *>(k_pool + base + (size_t)hw * CKV_D);
        const uint4 *vp = reinterpret_cast<const uint4 *>(v_pool + base + (size_t)hw * CKV_D);
        constexpr int kStep = 2 * CKV_D / 8;
        uint4 kraw[8], vraw[8];
        float mb[8], vb[8], qb[8];
        if (ntok == CKV_PAGE) {   // a full page: no per-row tests
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            kraw[j] = NC ? __ldg(kp + j * kStep) : kp[j * kStep];
            vraw[j] = NC ? __ldg(vp + j * kStep) : vp[j * kStep];
          }
          block_stats_rows16<true>(kraw, vraw, true, CKV_PAGE, lane, mb, vb, qb);
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const bool valid = hw + 2 * j < ntok;
            const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
            kraw[j] = valid ? (NC ? __ldg(kp + j * kStep) : kp[j * kStep]) : zero;
            vraw[j] = valid ? (NC ? __ldg(vp + j * kStep) : vp[j * kStep]) : zero;
          }
          block_stats_rows16(kraw, vraw, true, ntok, lane, mb, vb, qb);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) qb[i] += __shfl_xor_sync(0xffffffffu, qb[i], 16);
        combine_pages(na, km, m2, vs, ntok, mb, qb, vb);
      }
      // block_stats_finish adds the two half warps' squared deviations: the joined ones are already complete
#pragma unroll
      for (int i = 0; i < 8; ++i) sq[i] = hw == 0 ? m2[i] : 0.f;
    }
  }
  if constexpr (sizeof(T) != 2) {
  if (!done) {
    if constexpr (!NC) {
      // A block of several pages (32- or 64-token blocks) is read page after page, twice: when the caller works on
      // one block only (the append, the chunked prefill) the L2 is asked for all of its pages first, so that only
      // the first page costs a DRAM round trip.  (The build kernel asks for its next block itself.)
      if (npages > 1 && lane < npages) {
        const int phys = pt_row[b * P.ppb + lane];
        if (phys >= 0 && phys < P.num_pages) {
          const size_t off = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D;
          const unsigned bytes = CKV_PAGE * CKV_D * sizeof(T);
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(k_pool + off), "r"(bytes) : "memory");
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(v_pool + off), "r"(bytes) : "memory");
        }
      }
    }
    for (int pg = 0; pg < npages; ++pg) {
      const int phys = pt_row[b * P.ppb + pg];
      if (phys < 0 || phys >= P.num_pages) { bad = true; continue; }
      const size_t base = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8], c[8];
          load8<NC>(k_pool + base + (size_t)t * CKV_D, a);
          load8<NC>(v_pool + base + (size_t)t * CKV_D, c);
#pragma unroll
          for (int i = 0; i < 8; ++i) { ks[i] += a[i]; vs[i] += c[i]; }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      ks[i] += __shfl_xor_sync(0xffffffffu, ks[i], 16);
      vs[i] += __shfl_xor_sync(0xffffffffu, vs[i], 16);
      km[i] = ks[i] * inv;
      sq[i] = 0.f;
    }
    for (int pg = 0; pg < npages; ++pg) {
      const int phys = pt_row[b * P.ppb + pg];
      if (phys < 0 || phys >= P.num_pages) continue;
      const size_t base = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8];
          load8<NC>(k_pool + base + (size_t)t * CKV_D, a);
#pragma unroll
          for (int i = 0; i < 8; ++i) { const float dv = a[i] - km[i]; sq[i] = fmaf(dv, dv, sq[i]); }
        }
      }
    }
  }
  }
  if constexpr (ONEP) {
    if (!done) {   // not a one-page block after all: nothing is read, the summary is marked bad
      bad = true;
#pragma unroll
      for (int i = 0; i < 8; ++i) { km[i] = 0.f; sq[i] = 0.f; }
    }
  }
  block_stats_finish(P, b, fc, km, vs, sq, sq_smem, kmean_row, dbar_row, vmean_row, lane, bad);
}

// The same block routine for a caller whose time goes into instruction fetch rather than arithmetic (the tail
// warps of the scan launch run this code once per launch, next to a kernel that saturates DRAM): the rows of a
// page are brought into shared memory with asynchronous 16-byte copies issued from a rolled loop (all in flight
// together, no load waits for another), and both passes are rolled loops over the staged rows.  Same operations
// in the same order as block_stats_warp, hence the same bits; a third of its code.
// stage: 2 * CKV_PAGE * CKV_D * sizeof(T) bytes of shared memory owned by the calling warp, 16-byte aligned.
template <typename T>
__device__ __forceinline__ void block_stats_warp_staged(const CkvDev &P, const T *k_pool, const T *v_pool,
                                                        const int *pt_row, int h, int b, int cnt,
                                                        unsigned char *stage, float *sq_smem,
                                                        __nv_bfloat16 *kmean_row, float *dbar_row,
                                                        __nv_bfloat16 *vmean_row, int lane) {
  const int hw = lane >> 4, li = lane & 15;
  constexpr int kPageElems = CKV_PAGE * CKV_D;
  constexpr int kPieces = (int)(kPageElems * sizeof(T) / 16);   // 16-byte pieces of one head's K (or V) page
  const T *sk = reinterpret_cast<const T *>(stage), *sv = sk + kPageElems;
  const uint32_t stage_u32 = (uint32_t)__cvta_generic_to_shared(stage);
  float ks[8], vs[8], km[8], sq[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { ks[i] = 0.f; vs[i] = 0.f; }
  const int npages = (cnt + CKV_PAGE - 1) / CKV_PAGE;
  const float fc = (float)cnt, inv = 1.0f / fc;
  bool bad = false;
  auto stage_page = [&](int pg, bool with_v) -> bool {   // false: the page id is bad, nothing staged
    const int phys = pt_row[b * P.ppb + pg];
    if (phys < 0 || phys >= P.num_pages) return false;
    const size_t base = ((size_t)phys * P.Hkv + h) * kPageElems;
    const char *gk = reinterpret_cast<const char *>(k_pool + base), *gv = reinterpret_cast<const char *>(v_pool + base);
    const int n = with_v ? 2 * kPieces : kPieces;
#pragma unroll 1
    for (int p = lane; p < n; p += 32) {
      const char *src = p < kPieces ? gk + (size_t)p * 16 : gv + (size_t)(p - kPieces) * 16;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_u32 + (uint32_t)p * 16u), "l"(src) : "memory");
    }
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    return true;
  };
  if constexpr (sizeof(T) == 2) {
    // bf16 pages: every page is staged once and goes through its own two passes; several pages are joined as in
    // block_stats_warp (same operations, same order, same bits)
    float na = 0.f, m2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { km[i] = 0.f; m2[i] = 0.f; }
#pragma unroll 1
    for (int pg = 0; pg < npages; ++pg) {
      if (!stage_page(pg, true)) { bad = true; continue; }
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
      const float invp = 1.0f / (float)ntok;
      float kb[8], vb[8], mb[8], qb[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) { kb[i] = 0.f; vb[i] = 0.f; }
#pragma unroll 1
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8], c[8];
          load8<false>(sk + t * CKV_D + 8 * li, a);
          load8<false>(sv + t * CKV_D + 8 * li, c);
#pragma unroll
          for (int i = 0; i < 8; ++i) { kb[i] += a[i]; vb[i] += c[i]; }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        kb[i] += __shfl_xor_sync(0xffffffffu, kb[i], 16);
        vb[i] += __shfl_xor_sync(0xffffffffu, vb[i], 16);
        mb[i] = kb[i] * invp;
        qb[i] = 0.f;
      }
#pragma unroll 1
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8];
          load8<false>(sk + t * CKV_D + 8 * li, a);
#pragma unroll
          for (int i = 0; i < 8; ++i) { const float dv = a[i] - mb[i]; qb[i] = fmaf(dv, dv, qb[i]); }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) qb[i] += __shfl_xor_sync(0xffffffffu, qb[i], 16);
      combine_pages(na, km, m2, vs, ntok, mb, qb, vb);
      __syncwarp();   // the stage may be overwritten
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) sq[i] = hw == 0 ? m2[i] : 0.f;
  } else {
#pragma unroll 1
    for (int pg = 0; pg < npages; ++pg) {
      if (!stage_page(pg, true)) { bad = true; continue; }
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll 1
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8], c[8];
          load8<false>(sk + t * CKV_D + 8 * li, a);
          load8<false>(sv + t * CKV_D + 8 * li, c);
#pragma unroll
          for (int i = 0; i < 8; ++i) { ks[i] += a[i]; vs[i] += c[i]; }
        }
      }
      __syncwarp();   // the stage may be overwritten
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      ks[i] += __shfl_xor_sync(0xffffffffu, ks[i], 16);
      vs[i] += __shfl_xor_sync(0xffffffffu, vs[i], 16);
      km[i] = ks[i] * inv;
      sq[i] = 0.f;
    }
#pragma unroll 1
    for (int pg = 0; pg < npages; ++pg) {
      if (npages > 1 && !stage_page(pg, false)) continue;   // a one-page block is still staged from the first pass
      if (npages == 1 && bad) continue;
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll 1
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        if (t < ntok) {
          float a[8];
          load8<false>(sk + t * CKV_D + 8 * li, a);
#pragma unroll
          for (int i = 0; i < 8; ++i) { const float dv = a[i] - km[i]; sq[i] = fmaf(dv, dv, sq[i]); }
        }
      }
      __syncwarp();
    }
  }
  block_stats_finish(P, b, fc, km, vs, sq, sq_smem, kmean_row, dbar_row, vmean_row, lane, bad);
}

#endif  // CKV_BLOCKSTATS_CUH_
