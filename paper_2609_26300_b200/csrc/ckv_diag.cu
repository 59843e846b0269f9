// Exact per-block logit statistics (Eq. 3, App. B.1): a diagnostic pass over every key of the cache.
//
// For every (sequence, query head, block) the kernel reads the block's keys and produces
//   logZ_b  = log sum_{j in b} e^{z_j}         z_j = scale * q . k_j
//   zmean_b = mean_{j in b} z_j                (the logit of the block's mean key)
//   zvar_b  = population variance of the z_j   (the exact sigma_b^2 that Eq. 8 estimates)
// from which the exact block mass p_b, the exact compensation residual rho_b = p_b (1 - |b| e^{zmean_b} / Z_b)
// and the KL divergences of a selection follow by block-level arithmetic on the host.  It is not part of the
// decode step: it exists to measure how well the scorer ranks blocks on a given cache.
//
// One warp owns one block.  A key row (128 elements) is spread over the 16 lanes of a half warp, 8 coordinates
// per lane; the two half warps take alternate tokens.  Logits go through shared memory, then lanes take tokens
// and the three statistics are warp reductions (variance in two passes, around the mean).
#include "ckv_internal.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kMaxBlock = 64;   // tokens per block at most

template <typename T, int G>
__global__ void __launch_bounds__(kWarps * 32)
ckv_exact_blocks_kernel(CkvDev P, const T *__restrict__ q, const T *__restrict__ k_pool,
                        const int *__restrict__ page_table, const int *__restrict__ seq_lens,
                        float *__restrict__ logZ, float *__restrict__ zmean, float *__restrict__ zvar) {
  __shared__ float s_z[kWarps][G][kMaxBlock];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, hw = lane >> 4, li = lane & 15;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int N = max(min(seq_lens[s], P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) / P.bs;
  const int b = blockIdx.x * kWarps + warp;
  if (b >= X) return;   // whole warps leave; no CTA-wide barrier follows
  const int cnt = min(P.bs, N - b * P.bs);
  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;

  float qx[G][8];   // this lane's 8 coordinates of every head of the group
#pragma unroll
  for (int g = 0; g < G; ++g) load8<true>(q + ((size_t)s * P.Hq + h * G + g) * CKV_D + 8 * li, qx[g]);

  bool bad = false;
  const int npages = (cnt + CKV_PAGE - 1) / CKV_PAGE;
  for (int pg = 0; pg < npages; ++pg) {
    const int phys = pt_row[b * P.ppb + pg];
    const bool ok = phys >= 0 && phys < P.num_pages;
    bad |= !ok;
    const size_t base = ok ? ((size_t)phys * P.Hkv + h) * CKV_PAGE * CKV_D + 8 * li : 0;
    const int ntok = min(CKV_PAGE, cnt - pg * CKV_PAGE);
#pragma unroll
    for (int j = 0; j < CKV_PAGE / 2; ++j) {
      const int t = hw + 2 * j;   // uniform per half warp
      float a[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = 0.f;
      if (ok && t < ntok) load8<true>(k_pool + base + (size_t)t * CKV_D, a);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) d = fmaf(qx[g][i], a[i], d);
        d += __shfl_xor_sync(0xffffffffu, d, 8);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        if (li == 0 && t < ntok) s_z[warp][g][pg * CKV_PAGE + t] = ok ? d * P.scale : -CUDART_INF_F;
      }
    }
  }
  __syncwarp();
  if (bad && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);
  // lanes take tokens (two per lane for 64-token blocks)
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float z0 = lane < cnt ? s_z[warp][g][lane] : -CUDART_INF_F;
    const float z1 = lane + 32 < cnt ? s_z[warp][g][lane + 32] : -CUDART_INF_F;
    const float m = warp_max(fmaxf(z0, z1));
    const float se = warp_sum((lane < cnt ? expf(z0 - m) : 0.f) + (lane + 32 < cnt ? expf(z1 - m) : 0.f));
    const float mean = warp_sum((lane < cnt ? z0 : 0.f) + (lane + 32 < cnt ? z1 : 0.f)) / (float)cnt;
    const float d0 = lane < cnt ? z0 - mean : 0.f, d1 = lane + 32 < cnt ? z1 - mean : 0.f;
    const float var = warp_sum(d0 * d0 + d1 * d1) / (float)cnt;
    if (lane == 0) {
      const size_t o = ((size_t)s * P.Hq + h * G + g) * P.max_blocks + b;
      logZ[o] = m + logf(se);
      zmean[o] = mean;
      zvar[o] = var;
    }
  }
}

template <typename T>
cudaError_t launch_t(ckv_ctx *c, const void *q, const void *k_pool, const int *page_table, const int *seq_lens, dim3 grid,
                     float *logZ, float *zmean, float *zvar, cudaStream_t st) {
  const T *qp = (const T *)q, *kp = (const T *)k_pool;
  switch (c->dev.G) {
    case 1: ckv_exact_blocks_kernel<T, 1><<<grid, kWarps * 32, 0, st>>>(c->dev, qp, kp, page_table, seq_lens, logZ, zmean, zvar); break;
    case 2: ckv_exact_blocks_kernel<T, 2><<<grid, kWarps * 32, 0, st>>>(c->dev, qp, kp, page_table, seq_lens, logZ, zmean, zvar); break;
    case 4: ckv_exact_blocks_kernel<T, 4><<<grid, kWarps * 32, 0, st>>>(c->dev, qp, kp, page_table, seq_lens, logZ, zmean, zvar); break;
    case 8: ckv_exact_blocks_kernel<T, 8><<<grid, kWarps * 32, 0, st>>>(c->dev, qp, kp, page_table, seq_lens, logZ, zmean, zvar); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t ckv_launch_exact_blocks(ckv_ctx *c, const void *q, const void *k_pool, const int *page_table,
                                    const int *seq_lens, int batch, int max_len, float *logZ, float *zmean, float *zvar,
                                    cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int xmax = (max_len + P.bs - 1) / P.bs;
  if (xmax <= 0 || batch <= 0) return cudaSuccess;
  dim3 grid((xmax + kWarps - 1) / kWarps, batch * P.Hkv);
  c->launches++;
  if (c->layout.kv_dtype == CKV_BF16)
    return launch_t<__nv_bfloat16>(c, q, k_pool, page_table, seq_lens, grid, logZ, zmean, zvar, st);
  return launch_t<float>(c, q, k_pool, page_table, seq_lens, grid, logZ, zmean, zvar, st);
}
