// Block scores and selection for one unit per CTA (Eq. 9-11).
//
//   phat_{g,b} = exp(l_{g,b} - M_g) / sum_c exp(l_{g,c} - M_g),  M_g = max_c l_{g,c}   (Eq. 9, all blocks)
//   S_b        = sum_g phat_{g,b} sigma_hat^2_{g,b}                                      (Eq. 10)
//   S          = F  u  TopK_{K-|F|} { S_b : b not in F },  ids ascending                (Eq. 11)
// F = first `sink` and last `recent` blocks.  Equal scores go to the lower block id.  The K-th
// largest score is found exactly with a most-significant-digit-first radix select on the fp32 bit
// patterns (scores are >= 0, so unsigned order is numeric order); ids come out in position order
// from a prefix sum over selection flags.
#include "ckv_internal.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kSmemKeys = 24576;   // keys cached in shared memory (96 KB); longer units re-read global scores

__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_tot, int *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    warp_tot[lane] = winc - w;
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  const int res = warp_tot[warp] + inc - v;
  __syncthreads();
  return res;
}

template <int G>
__global__ void __launch_bounds__(kThreads) ckv_select_kernel(CkvDev P, const int *__restrict__ seq_lens, int kcap,
                                                              int *__restrict__ sel_ids, int *__restrict__ sel_cnt) {
  extern __shared__ uint32_t skeys[];
  __shared__ float s_red[32][G];
  __shared__ float s_M[G], s_invL[G];
  __shared__ int s_hist[256];
  __shared__ int s_wtot[32];
  __shared__ int s_total, s_digit, s_remaining;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x, s = unit / P.Hkv;
  const int N = min(seq_lens[s], P.max_blocks * P.bs);
  const int X = (N + P.bs - 1) / P.bs;
  int *ids = sel_ids + (size_t)unit * kcap;
  const int K = min(kcap, X);
  if (X <= kcap) {   // every block is selected: the step is dense attention
    for (int b = tid; b < kcap; b += kThreads) ids[b] = b < X ? b : -1;
    if (tid == 0) sel_cnt[unit] = X;
    // scores are still produced below for callers that read them
  }
  const float2 *ls = P.ls + (size_t)unit * P.max_blocks * G;
  float *scores = P.scores + (size_t)unit * P.max_blocks;

  // M_g
  float m[G];
#pragma unroll
  for (int g = 0; g < G; ++g) m[g] = -CUDART_INF_F;
  for (int b = tid; b < X; b += kThreads)
#pragma unroll
    for (int g = 0; g < G; ++g) m[g] = fmaxf(m[g], ls[(size_t)b * G + g].x);
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = warp_max(m[g]);
    if (lane == 0) s_red[warp][g] = m[g];
  }
  __syncthreads();
  if (tid < G) {
    float v = -CUDART_INF_F;
    for (int w = 0; w < 32; ++w) v = fmaxf(v, s_red[w][tid]);
    s_M[tid] = v;
  }
  __syncthreads();
  // L_g = sum_b exp(l - M)
  float l[G];
#pragma unroll
  for (int g = 0; g < G; ++g) { m[g] = s_M[g]; l[g] = 0.f; }
  for (int b = tid; b < X; b += kThreads)
#pragma unroll
    for (int g = 0; g < G; ++g) l[g] += expf(ls[(size_t)b * G + g].x - m[g]);
  __syncthreads();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    l[g] = warp_sum(l[g]);
    if (lane == 0) s_red[warp][g] = l[g];
  }
  __syncthreads();
  if (tid < G) {
    float v = 0.f;
    for (int w = 0; w < 32; ++w) v += s_red[w][tid];
    s_invL[tid] = 1.0f / v;
  }
  __syncthreads();
  // S_b
  const bool cached = X <= kSmemKeys;
  bool nonfinite = false;
  for (int b = tid; b < X; b += kThreads) {
    float sc = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float2 v = ls[(size_t)b * G + g];
      sc = fmaf(expf(v.x - m[g]) * s_invL[g], v.y, sc);
    }
    if (!(sc >= 0.f) || sc > 3.0e38f) { nonfinite = true; sc = 0.f; }
    scores[b] = sc;
    if (cached) skeys[b] = __float_as_uint(sc);
  }
  if (nonfinite) atomicOr(P.status, CKV_DEV_NONFINITE);
  __syncthreads();   // scores[] written by this CTA are read back below (same CTA: visible after the barrier)
  if (X <= kcap) return;

  const uint32_t *keys = cached ? skeys : reinterpret_cast<const uint32_t *>(scores);
  const int n_tail = min(P.recent, X);
  auto mandatory = [&](int b) { return b < P.sink || b >= X - n_tail; };
  int nF = min(P.sink, X) + n_tail;
  if (P.sink + n_tail > X) nF = X;
  const int Kr = K - nF;   // blocks to rank in (host guarantees K >= sink + recent when K < X)

  uint32_t prefix = 0, pmask = 0;
  if (tid == 0) s_remaining = Kr;
  __syncthreads();
  if (Kr > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) s_hist[tid] = 0;
      __syncthreads();
      for (int b = tid; b < X; b += kThreads) {
        if (mandatory(b)) continue;
        const uint32_t k = keys[b];
        if ((k & pmask) == prefix) atomicAdd(&s_hist[(k >> shift) & 255], 1);
      }
      __syncthreads();
      if (warp == 0) {
        // digits from high to low: find the digit where the running count reaches `remaining`
        const int remaining = s_remaining;
        int cnt8 = 0;   // lane covers digits 255 - 8*lane - j, j = 0..7
        int c[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = s_hist[255 - 8 * lane - j]; cnt8 += c[j]; }
        int inc = cnt8;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += t;
        }
        int before = inc - cnt8;   // keys with a higher digit than this lane's range
        if (before < remaining && inc >= remaining) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (before < remaining && before + c[j] >= remaining) {
              s_digit = 255 - 8 * lane - j;
              s_remaining = remaining - before;
              before = remaining;   // stop
            } else {
              before += c[j];
            }
          }
        }
      }
      __syncthreads();
      prefix |= (uint32_t)s_digit << shift;
      pmask |= 255u << shift;
      __syncthreads();
    }
  }
  const uint32_t thr = prefix;          // bit pattern of the Kr-th largest ranked score
  const int need_eq = s_remaining;      // how many blocks scoring exactly thr are taken (lowest ids first)

  // ordered emission: thread t owns a contiguous range of blocks
  const int per = (X + kThreads - 1) / kThreads;
  const int b0 = min(tid * per, X), b1 = min(b0 + per, X);
  int c_eq = 0;
  if (Kr > 0)
    for (int b = b0; b < b1; ++b) c_eq += (!mandatory(b) && keys[b] == thr) ? 1 : 0;
  int eq_rank = block_exclusive_scan(c_eq, s_wtot, &s_total);
  int c_sel = 0;
  {
    int e = eq_rank;
    for (int b = b0; b < b1; ++b) {
      bool sel = mandatory(b);
      if (!sel && Kr > 0) {
        const uint32_t k = keys[b];
        if (k > thr) sel = true;
        else if (k == thr) { sel = e < need_eq; ++e; }
      }
      c_sel += sel ? 1 : 0;
    }
  }
  int pos = block_exclusive_scan(c_sel, s_wtot, &s_total);
  const int total = s_total;
  {
    int e = eq_rank;
    for (int b = b0; b < b1; ++b) {
      bool sel = mandatory(b);
      if (!sel && Kr > 0) {
        const uint32_t k = keys[b];
        if (k > thr) sel = true;
        else if (k == thr) { sel = e < need_eq; ++e; }
      }
      if (sel) { if (pos < kcap) ids[pos] = b; ++pos; }
    }
  }
  for (int i = total + tid; i < kcap; i += kThreads) ids[i] = -1;
  if (tid == 0) sel_cnt[unit] = min(total, kcap);
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, const int *seq_lens, int units, int kcap, int *sel_ids, int *sel_cnt,
                     cudaStream_t st) {
  const size_t smem = (size_t)kSmemKeys * sizeof(uint32_t);
  ckv_select_kernel<G><<<units, kThreads, smem, st>>>(c->dev, seq_lens, kcap, sel_ids, sel_cnt);
  return cudaGetLastError();
}

template <int G>
cudaError_t configure_g() {
  return cudaFuncSetAttribute(ckv_select_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)(kSmemKeys * sizeof(uint32_t)));
}

}  // namespace

// Opt in to the dynamic shared memory the selection kernel needs, on the current device.
cudaError_t ckv_configure_kernels() {
  cudaError_t e = configure_g<1>();
  if (e == cudaSuccess) e = configure_g<2>();
  if (e == cudaSuccess) e = configure_g<4>();
  if (e == cudaSuccess) e = configure_g<8>();
  return e;
}

cudaError_t ckv_launch_select(ckv_ctx *c, const int *seq_lens, int batch, int kcap, int *sel_ids, int *sel_cnt,
                              cudaStream_t st) {
  const int units = batch * c->dev.Hkv;
  c->launches++;
  switch (c->dev.G) {
    case 1: return launch_g<1>(c, seq_lens, units, kcap, sel_ids, sel_cnt, st);
    case 2: return launch_g<2>(c, seq_lens, units, kcap, sel_ids, sel_cnt, st);
    case 4: return launch_g<4>(c, seq_lens, units, kcap, sel_ids, sel_cnt, st);
    case 8: return launch_g<8>(c, seq_lens, units, kcap, sel_ids, sel_cnt, st);
  }
  return cudaErrorInvalidValue;
}
