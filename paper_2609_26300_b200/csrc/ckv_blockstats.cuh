// The block-summary routine shared by the prefill-time build, the per-token append and the chunked prefill
// (Sec. 4.1-4.2, Eq. 8 right half): one warp works out mean key, grouped variance and mean value of one block.
//
// A token row (128 elements) is spread over the 16 lanes of a half warp, 8 consecutive coordinates per lane (one
// 16-byte load for bf16); the two half warps take alternate rows.  Means and squared deviations are accumulated in
// fp32 in two passes (mean first, then deviations from it).  Every caller runs this same code, so a block's
// summary has the same bits whichever way it was produced.
#ifndef CKV_BLOCKSTATS_CUH_
#define CKV_BLOCKSTATS_CUH_
#include "ckv_internal.cuh"

// NC: the pools are read-only for the whole kernel (loads may use the non-coherent path).
// SMALL: compact code for callers that are bound by memory latency and share their kernel with a hot loop whose
// instructions should stay cached: loops are not unrolled and the register-resident one-page path is left out
// (the general path performs the same operations in the same order, hence the same bits).
// sq_smem: 128 floats of shared memory owned by the calling warp.
template <typename T, bool NC, bool SMALL = false>
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
  const float fc = (float)cnt;
  float km[8], sq[8];
  bool done = false;
  if constexpr (sizeof(T) == 2 && !SMALL) {
    if (npages == 1) {
      // One page of bf16 rows (every block of the default 16-token layout): the key rows stay in registers between
      // the two passes, so the cache is read exactly once.  Same operations in the same order as the general path
      // below (rows that do not exist contribute exact zeros), hence the same bits.
      done = true;
      const int phys = pt_row[b * P.ppb];
      const bool ok = phys >= 0 && phys < P.num_pages;
      bad = !ok;
      const size_t base = ok ? ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li : 0;
      uint4 kraw[8], vraw[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = hw + 2 * j;
        const bool valid = ok && t < cnt;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const uint4 *kp = reinterpret_cast<const uint4 *>(k_pool + base + (size_t)t * CKV_D);
        const uint4 *vp = reinterpret_cast<const uint4 *>(v_pool + base + (size_t)t * CKV_D);
        kraw[j] = valid ? (NC ? __ldg(kp) : *kp) : zero;
        vraw[j] = valid ? (NC ? __ldg(vp) : *vp) : zero;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (ok && hw + 2 * j < cnt) {
          float a[8], c[8];
          bf16x8_to_float(kraw[j], a);
          bf16x8_to_float(vraw[j], c);
#pragma unroll
          for (int i = 0; i < 8; ++i) { ks[i] += a[i]; vs[i] += c[i]; }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ks[i] += __shfl_xor_sync(0xffffffffu, ks[i], 16);
        vs[i] += __shfl_xor_sync(0xffffffffu, vs[i], 16);
        km[i] = ks[i] / fc;
        sq[i] = 0.f;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (ok && hw + 2 * j < cnt) {
          float a[8];
          bf16x8_to_float(kraw[j], a);
#pragma unroll
          for (int i = 0; i < 8; ++i) { const float dv = a[i] - km[i]; sq[i] = fmaf(dv, dv, sq[i]); }
        }
      }
    }
  }
  if (!done) {
    for (int pg = 0; pg < npages; ++pg) {
      const int phys = pt_row[b * P.ppb + pg];
      if (phys < 0 || phys >= P.num_pages) { bad = true; continue; }
      const size_t base = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll(SMALL ? 1 : 8)
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
      km[i] = ks[i] / fc;
      sq[i] = 0.f;
    }
    for (int pg = 0; pg < npages; ++pg) {
      const int phys = pt_row[b * P.ppb + pg];
      if (phys < 0 || phys >= P.num_pages) continue;
      const size_t base = ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li;
      const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll(SMALL ? 1 : 8)
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
#pragma unroll
  for (int i = 0; i < 8; ++i) sq[i] += __shfl_xor_sync(0xffffffffu, sq[i], 16);
  if (hw == 0) {
    store_split8(kmean_row, li, b, km, P.row_elems == CKV_ROW_ELEMS);
    if (P.r == CKV_D) {
      // one group per coordinate: the variance row has the mean rows' layout (split bf16 pairs, swizzled chunks),
      // so that the scan can project it with the same tensor-core product as the mean keys
      float dv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) dv[i] = sq[i] / fc;
      store_split8(reinterpret_cast<__nv_bfloat16 *>(dbar_row), li, b, dv);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) sq_smem[8 * li + i] = sq[i];
    }
  } else {
    float vm[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) vm[i] = vs[i] / fc;
    store_split8(vmean_row, li, b, vm, P.row_elems == CKV_ROW_ELEMS);
  }
  __syncwarp();
  // grouped variance: average of the per-coordinate population variances of each group (Eq. 8)
  const int gs = CKV_D / P.r;
  for (int t = lane; t < P.r && P.r != CKV_D; t += 32) {
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
  if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);
}

#endif  // CKV_BLOCKSTATS_CUH_
