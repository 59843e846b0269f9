// Summary scan: one streaming pass over every block summary of a unit (Eq. 8-9 and the
// compensation sums of Eq. 12).
//
// For every block b and query head g of the unit the pass computes
//   zbar_{g,b}        = q_g . kbar_b * scale                      (block-mean logit, Sec. 4.1)
//   sigma_hat^2_{g,b} = scale^2 sum_t w_{g,t} Dbar_{b,t}         (Eq. 8 with 1/d = scale^2, w_{g,t} = sum_{i in G_t} q_{g,i}^2)
//   l_{g,b}           = log|b| + zbar + sigma_hat^2 / 2           (log of the numerator of Eq. 9)
// and stores (l, sigma_hat^2) for the selection kernel.  In the same pass it accumulates the
// mean-compensation terms of Eq. 12 over ALL blocks,  sum_b |b| e^{zbar} vbar_b  and
// sum_b |b| e^{zbar},  as online-softmax partials; the terms of the blocks that end up selected
// are taken out again by the attention kernel.  That way kbar, Dbar and vbar are each read
// from HBM exactly once per decode step.
//
// Mapping: 16 lanes share one block row (128 fp32 = 32 float4; lane li takes float4 li and li+16,
// so each load instruction of a half warp covers 256 contiguous bytes); a warp does two blocks at
// a time and the 8 warps of a CTA cover 16 consecutive blocks per iteration.  Each lane keeps its
// 8 coordinates of q (all G heads) and of the G output accumulators in registers.
#include "ckv_internal.cuh"

namespace {

template <int G> struct Log2 { static constexpr int v = 1 + Log2<G / 2>::v; };
template <> struct Log2<1> { static constexpr int v = 0; };

template <int G, typename QT>
__global__ void __launch_bounds__(256, (G <= 4) ? 2 : 1)
ckv_scan_kernel(CkvDev P, const QT *__restrict__ q, const int *__restrict__ seq_lens, int chunk) {
  constexpr int SH = 4 - Log2<G>::v;   // lane (g << SH) of a half warp owns head g after the reduction
  __shared__ float sq[G][CKV_D];
  __shared__ __align__(16) float sw[CKV_D][G];
  __shared__ __align__(16) float red[8][G][CKV_PART_STRIDE];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 4, li = lane & 15;
  const int unit = blockIdx.y, s = unit / P.Hkv, h = unit % P.Hkv;
  const int N = min(seq_lens[s], P.max_blocks * P.bs);
  const int X = (N + P.bs - 1) / P.bs;
  const int c0 = blockIdx.x * chunk;
  const int c1 = min(c0 + chunk, X);
  float *part = P.comp_part + ((size_t)unit * CKV_MAX_CHUNKS + blockIdx.x) * G * CKV_PART_STRIDE;
  if (c0 >= X) {   // nothing here: leave an empty partial
    if (tid < G) { part[tid * CKV_PART_STRIDE] = -CUDART_INF_F; part[tid * CKV_PART_STRIDE + 1] = 0.f; }
    return;
  }

  for (int idx = tid; idx < G * CKV_D; idx += 256)
    sq[idx / CKV_D][idx % CKV_D] = to_float(q[((size_t)s * P.Hq + h * G) * CKV_D + idx]);
  __syncthreads();
  for (int idx = tid; idx < P.r * G; idx += 256) {
    const int t = idx / G, g = idx % G;
    float w = 0.f;
    for (int i = 0; i < CKV_D; ++i)
      if (group_of(i, P.r, P.glayout) == t) w = fmaf(sq[g][i], sq[g][i], w);
    sw[t][g] = w;
  }
  __syncthreads();

  float qr[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      qr[g][i] = sq[g][4 * li + i] * P.scale;
      qr[g][4 + i] = sq[g][64 + 4 * li + i] * P.scale;
    }

  const size_t row0 = (size_t)unit * P.max_blocks;
  const float4 *km4 = reinterpret_cast<const float4 *>(P.kmean + row0 * CKV_D);
  const float4 *vm4 = reinterpret_cast<const float4 *>(P.vmean + row0 * CKV_D);
  const float *db = P.dbar + row0 * P.r;
  float2 *ls = P.ls + row0 * G;

  float acc[G][8], m_ref[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_ref[g] = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;
  }
  float m_my = -CUDART_INF_F, l_my = 0.f;
  const int myg = li >> SH;
  const float log_bs = logf((float)P.bs);
  const float log_last = logf((float)(N - (X - 1) * P.bs));
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

  int b = c0 + warp * 2 + gid;
  float4 k0 = zero4, k1 = zero4, v0 = zero4, v1 = zero4;
  if (b < c1) {
    k0 = __ldg(km4 + (size_t)b * 32 + li); k1 = __ldg(km4 + (size_t)b * 32 + 16 + li);
    v0 = __ldg(vm4 + (size_t)b * 32 + li); v1 = __ldg(vm4 + (size_t)b * 32 + 16 + li);
  }
  for (int base = c0; base < c1; base += 16) {
    const bool valid = b < c1;
    const float kk[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
    const float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    const int bn = b + 16;
    if (bn < c1) {   // prefetch the next rows while this one is being reduced
      k0 = __ldg(km4 + (size_t)bn * 32 + li); k1 = __ldg(km4 + (size_t)bn * 32 + 16 + li);
      v0 = __ldg(vm4 + (size_t)bn * 32 + li); v1 = __ldg(vm4 + (size_t)bn * 32 + 16 + li);
    }
    float red_v[2 * G];
#pragma unroll
    for (int g = 0; g < G; ++g) { red_v[2 * g] = 0.f; red_v[2 * g + 1] = 0.f; }
    if (valid) {
      for (int t = li; t < P.r; t += 16) {
        const float dv = __ldg(db + (size_t)b * P.r + t);
#pragma unroll
        for (int g = 0; g < G; ++g) red_v[2 * g + 1] = fmaf(sw[t][g], dv, red_v[2 * g + 1]);
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float z = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) z = fmaf(qr[g][i], kk[i], z);
      red_v[2 * g] = z;
    }
    reduce16<2 * G, 2>(red_v, li);
    const float zbar = red_v[0];
    const float sig = red_v[1] * (P.scale * P.scale);   // Eq. 8's 1/d is the squared logit scale
    const float logc = (b == X - 1) ? log_last : log_bs;
    const float ell = logc + zbar + 0.5f * sig;
    if (valid && (li & ((1 << SH) - 1)) == 0) ls[(size_t)b * G + myg] = make_float2(ell, sig);
    // compensation weight of this block for head myg: |b| e^{zbar}, in log2 units
    const float zl2 = valid ? (zbar + logc) * kLog2e : -CUDART_INF_F;
    if (__any_sync(0xffffffffu, zl2 > m_my + CKV_RESCALE_SLACK)) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float cand = __shfl_sync(0xffffffffu, zl2, (lane & 16) | (g << SH));
        if (cand > m_ref[g]) {
          const float sc = exp2_diff(m_ref[g], cand);
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[g][i] *= sc;
          if (myg == g) { l_my *= sc; m_my = cand; }
          m_ref[g] = cand;
        }
      }
    }
    const float wt = valid ? exp2f(zl2 - m_my) : 0.f;
    l_my += wt;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float wg = __shfl_sync(0xffffffffu, wt, (lane & 16) | (g << SH));
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[g][i] = fmaf(wg, vv[i], acc[g][i]);
    }
    b = bn;
  }

  // fold the two half warps, then the 8 warps, into one partial per head
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float mo = __shfl_xor_sync(0xffffffffu, m_ref[g], 16);
    const float mn = fmaxf(m_ref[g], mo);
    const float sc = exp2_diff(m_ref[g], mn);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float a = acc[g][i] * sc;
      acc[g][i] = a + __shfl_xor_sync(0xffffffffu, a, 16);
    }
    float lg = (myg == g) ? l_my * sc : 0.f;
    lg += __shfl_xor_sync(0xffffffffu, lg, 16);
    if (myg == g) l_my = lg;
    m_ref[g] = mn;
  }
  if (gid == 0) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float *r = red[warp][g];
      *reinterpret_cast<float4 *>(r + 4 + 4 * li) = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
      *reinterpret_cast<float4 *>(r + 4 + 64 + 4 * li) = make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]);
      if (li == (g << SH)) { r[0] = m_ref[g]; r[1] = l_my; }
    }
  }
  __syncthreads();
  for (int idx = tid; idx < G * CKV_D; idx += 256) {
    const int g = idx / CKV_D, i = idx % CKV_D;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < 8; ++w) M = fmaxf(M, red[w][g][0]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float sc = exp2_diff(red[w][g][0], M);
      num = fmaf(red[w][g][4 + i], sc, num);
      den = fmaf(red[w][g][1], sc, den);
    }
    part[g * CKV_PART_STRIDE + 4 + i] = num;
    if (i == 0) { part[g * CKV_PART_STRIDE] = M; part[g * CKV_PART_STRIDE + 1] = den; }
  }
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, const void *q, const int *seq_lens, dim3 grid, int chunk, cudaStream_t st) {
  if (c->layout.kv_dtype == CKV_BF16)
    ckv_scan_kernel<G, __nv_bfloat16><<<grid, 256, 0, st>>>(c->dev, (const __nv_bfloat16 *)q, seq_lens, chunk);
  else
    ckv_scan_kernel<G, float><<<grid, 256, 0, st>>>(c->dev, (const float *)q, seq_lens, chunk);
  return cudaGetLastError();
}

}  // namespace

cudaError_t ckv_launch_scan(ckv_ctx *c, const void *q, const int *seq_lens, int batch, int max_len,
                            int *n_chunks_out, cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int units = batch * P.Hkv;
  const int xmax = (max_len + P.bs - 1) / P.bs;
  // about four CTAs per SM overall, at least 32 blocks per CTA, at most CKV_MAX_CHUNKS chunks per unit
  int n_chunks = (148 * 4 + units - 1) / units;
  n_chunks = max(1, min(n_chunks, min(CKV_MAX_CHUNKS, (xmax + 31) / 32)));
  int chunk = (xmax + n_chunks - 1) / n_chunks;
  chunk = (chunk + 15) / 16 * 16;
  n_chunks = (xmax + chunk - 1) / chunk;
  *n_chunks_out = n_chunks;
  dim3 grid(n_chunks, units);
  c->launches++;
  switch (P.G) {
    case 1: return launch_g<1>(c, q, seq_lens, grid, chunk, st);
    case 2: return launch_g<2>(c, q, seq_lens, grid, chunk, st);
    case 4: return launch_g<4>(c, q, seq_lens, grid, chunk, st);
    case 8: return launch_g<8>(c, q, seq_lens, grid, chunk, st);
  }
  return cudaErrorInvalidValue;
}
