// Block scores and selection for one unit per CTA (Eq. 9-11).
//
//   phat_{g,b} = exp(l_{g,b} - M_g) / L_g,  L_g = sum_c exp(l_{g,c} - M_g)      (Eq. 9, over all blocks)
//   S_b        = sum_g phat_{g,b} sigma_hat^2_{g,b}                              (Eq. 10)
//   S          = F  u  TopK_{K-|F|} { S_b : b not in F },  ids ascending        (Eq. 11)
// F = first `sink` and last `recent` blocks.  Equal scores go to the lower block id.
//
// The scan kernel leaves, per head and block, u_{g,b} = log2(e^{l_{g,b}} sigma_hat^2_{g,b}) (4 bytes) and the
// normalisers (M_g, L_g) as per-CTA partials, so S_b = sum_g 2^{u_{g,b} - M_g} / L_g and every term is read
// once.  The normaliser loads are issued before the (much larger) batch of u loads, which would otherwise sit in
// front of them in the memory pipeline.  The K-th largest score is found exactly with a most-significant-
// digit-first radix select on the fp32 bit patterns (scores are >= 0, so unsigned order is numeric order): a
// 4096-bin histogram of the top 12 bits, built while the scores are computed, then a direct ranking of the blocks
// in the bin that holds the threshold (falling back to 12 + 8 more bits on heavy ties); ids come out in position
// order from a prefix sum over selection flags.
#include "ckv_internal.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kSmemKeys = 24576;   // keys cached in shared memory (96 KB); longer units re-read global scores
constexpr int kBins = 4096;

// Exclusive prefix sum of one int per thread over the CTA; *total receives the sum.
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
    const int w = warp_tot[lane];
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
                                                              int scan_grid, int units, int *__restrict__ sel_ids,
                                                              int *__restrict__ sel_cnt) {
  extern __shared__ uint32_t skeys[];
  __shared__ int s_hist[kBins];
  __shared__ float s_M[G], s_invL[G];
  __shared__ int s_wtot[32];
  __shared__ int s_total, s_digit, s_remaining, s_ncand;
  __shared__ int s_cand[kThreads];
  __shared__ uint32_t s_candk[kThreads];   // the candidates' keys, so that the ranking loop reads no key through an id

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x, s = ckv_div_hkv(P, unit);
  const int N = max(min(seq_lens[s], P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) >> P.lg_bs;
  int *ids = sel_ids + (size_t)unit * kcap;
  const int K = min(kcap, X);
  if (X <= kcap) {   // every block is selected: the step is dense attention
    for (int b = tid; b < kcap; b += kThreads) ids[b] = b < X ? b : -1;
    if (tid == 0) sel_cnt[unit] = X;
    if (X == 0) return;
    // scores are still produced below for callers that read them
  }

  // ---- normalisers of Eq. 9: M_g, L_g from the scan partials of this unit (entries (c + unit) * W + w, c in
  // [cfirst, cfirst + ccount)).  Warp g works them out for head g; its loads are issued before the much larger
  // batch of score-term loads below, which would otherwise sit in front of them in the memory pipeline. ----
  if (tid == 0) s_ncand = 0;
  for (int i = tid; i < kBins; i += kThreads) s_hist[i] = 0;   // the first radix pass fills it while scoring
  float pm[4], pl[4];
  const float *cp = nullptr;
  int n_part = 0;
  const size_t pstep = (size_t)G * CKV_PART_STRIDE;
  if (warp < G) {
    int efirst;
    unit_scan_entries(P, CkvClampedLens{seq_lens, P.max_blocks * P.bs}, units, unit, scan_grid, lane, efirst, n_part);
    cp = P.comp_part + ((size_t)efirst * G + warp) * CKV_PART_STRIDE;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = lane + 32 * k;
      pm[k] = i < n_part ? cp[i * pstep] : -CUDART_INF_F;
      pl[k] = i < n_part ? cp[i * pstep + 2] : 0.f;
    }
  }
  // the first batch of (l, sigma^2) loads does not depend on the normalisers: it is in flight while they are reduced
  constexpr int NB = G >= 8 ? 4 : 8;   // blocks per thread and batch (their loads are in flight together)
  const float *lu = P.lu + (size_t)unit * P.max_blocks * G;   // log2(e^l sigma^2) per head and block, from the scan
  float *scores = P.scores + (size_t)unit * P.max_blocks;
  float v[NB][G];
  auto load_batch = [&](int base) {
#pragma unroll
    for (int j = 0; j < NB; ++j) {
      const int b = base + j * kThreads + tid;
      if (b < X) {
#pragma unroll
        for (int g = 0; g < G; ++g) v[j][g] = lu[(size_t)g * P.max_blocks + b];   // head-major: coalesced per head
      }
    }
  };
  load_batch(0);
  if (warp < G) {
    float m = fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3]));
    for (int i = lane + 128; i < n_part; i += 32) m = fmaxf(m, cp[i * pstep]);
    m = warp_max(m);
    float l = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) l = fmaf(pl[k], exp2_diff(pm[k], m), l);
    for (int i = lane + 128; i < n_part; i += 32) l = fmaf(cp[i * pstep + 2], exp2_diff(cp[i * pstep], m), l);
    l = warp_sum(l);
    if (lane == 0) { s_M[warp] = m; s_invL[warp] = 1.0f / l; }
  }
  __syncthreads();

  // ---- S_b ----
  float Mg[G], iL[G];
#pragma unroll
  for (int g = 0; g < G; ++g) { Mg[g] = s_M[g]; iL[g] = s_invL[g]; }
  const int n_tail = min(P.recent, X);
  auto mandatory = [&](int b) { return b < P.sink || b >= X - n_tail; };
  int nF = min(P.sink, X) + n_tail;
  if (P.sink + n_tail > X) nF = X;
  const int Kr = K - nF;   // blocks to rank in (the host guarantees K >= sink + recent when K < X)
  if (tid == 0) { s_remaining = Kr; s_total = 0; }   // read after the barrier that follows the scoring loop
  const bool hist0 = X > kcap && Kr > 0;   // the first radix pass (top 12 bits of every ranked key) is built on the fly
  const bool cached = X <= kSmemKeys;
  bool nonfinite = false;
  for (int base = 0; base < X; base += NB * kThreads) {
    if (base > 0) load_batch(base);
#pragma unroll
    for (int j = 0; j < NB; ++j) {
      const int b = base + j * kThreads + tid;
      if (b < X) {
        float sc = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) sc = fmaf(fast_exp2(v[j][g] - Mg[g]), iL[g], sc);
        if (!(sc >= 0.f) || sc > 3.0e38f) { nonfinite = true; sc = 0.f; }
        scores[b] = sc;
        if (cached) skeys[b] = __float_as_uint(sc);
        if (hist0 && !mandatory(b)) atomicAdd(&s_hist[__float_as_uint(sc) >> 20], 1);
      }
    }
  }
  if (nonfinite) atomicOr(P.status, CKV_DEV_NONFINITE);
  __syncthreads();   // scores[] written by this CTA are read back below (same CTA: visible after the barrier)
  if (X <= kcap) return;

  const uint32_t *keys = cached ? skeys : reinterpret_cast<const uint32_t *>(scores);

  // ---- the Kr-th largest ranked score: one 12-bit radix pass, then either a direct ranking of the blocks in the
  //      digit bin that holds it (the usual case: a few dozen blocks) or the remaining radix passes ----
  uint32_t prefix = 0, pmask = 0;
  int eq_total = 0;   // blocks scoring exactly the threshold (radix path)
  bool ranked = false;   // direct-ranking path taken: chosen blocks carry the sign bit in skeys
  if (Kr > 0) {
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 20 : (pass == 1 ? 8 : 0);
      const int bins = pass == 2 ? 256 : kBins;
      if (pass > 0) {   // pass 0's histogram was built while the scores were computed
        for (int i = tid; i < bins; i += kThreads) s_hist[i] = 0;
        __syncthreads();
        for (int b = tid; b < X; b += kThreads) {
          if (mandatory(b)) continue;
          const uint32_t k = keys[b];
          if ((k & pmask) == prefix) atomicAdd(&s_hist[(k >> shift) & (bins - 1)], 1);
        }
        __syncthreads();
      }
      // thread t owns the four bins bins-1-4t ... bins-4-4t (highest digits first)
      int c[4], c4 = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int bin = bins - 1 - 4 * tid - j;
        c[j] = bin >= 0 ? s_hist[bin] : 0;
        c4 += c[j];
      }
      const int remaining = s_remaining;
      int before = block_exclusive_scan(c4, s_wtot, &s_total);   // keys with a higher digit than this thread's bins
      if (before < remaining && before + c4 >= remaining) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (before < remaining && before + c[j] >= remaining) {
            s_digit = bins - 1 - 4 * tid - j;
            s_remaining = remaining - before;
            s_total = c[j];
            before = remaining;   // stop
          } else {
            before += c[j];
          }
        }
      }
      __syncthreads();
      prefix |= (uint32_t)s_digit << shift;
      pmask |= (uint32_t)(bins - 1) << shift;
      eq_total = s_total;
      const int take = s_remaining;
      __syncthreads();
      if (pass == 0 && cached && eq_total <= kThreads) {
        // rank the bin's blocks by (score descending, id ascending) and mark the first `take`
        for (int b = tid; b < X; b += kThreads) {
          if (mandatory(b)) continue;
          const uint32_t k = keys[b];
          if ((k & pmask) == prefix) {
            const int slot = atomicAdd(&s_ncand, 1);
            s_cand[slot] = b;
            s_candk[slot] = k;
          }
        }
        __syncthreads();
        const int nc = s_ncand;
        bool chosen = false;
        int myb = -1;
        if (tid < nc) {
          myb = s_cand[tid];
          const uint32_t mk = s_candk[tid];
          int rank = 0;
#pragma unroll 8
          for (int j = 0; j < nc; ++j) {
            const int ob = s_cand[j];
            const uint32_t ok = s_candk[j];
            rank += (ok > mk || (ok == mk && ob < myb)) ? 1 : 0;
          }
          chosen = rank < take;
        }
        __syncthreads();   // every rank is computed before any key is marked
        if (chosen) skeys[myb] |= 0x80000000u;
        __syncthreads();
        ranked = true;
        break;
      }
    }
  }
  const uint32_t thr = prefix;          // radix path: bit pattern of the Kr-th largest ranked score
  const int need_eq = s_remaining;      // ... and how many blocks scoring exactly thr are taken (lowest ids first)
  const uint32_t digit0 = prefix >> 20; // ranking path: the 12-bit digit of the bin that was ranked

  // ---- ordered emission: thread t owns a contiguous range of blocks (odd length: conflict-free smem reads) ----
  const int per = ((X + kThreads - 1) / kThreads) | 1;
  const int b0 = min(tid * per, X), b1 = min(b0 + per, X);
  int eq_rank = 0;
  const bool all_eq = need_eq >= eq_total;   // every block at the threshold is taken: no rank among ties needed
  if (Kr > 0 && !ranked && !all_eq) {
    int c_eq = 0;
    for (int b = b0; b < b1; ++b) c_eq += (!mandatory(b) && keys[b] == thr) ? 1 : 0;
    eq_rank = block_exclusive_scan(c_eq, s_wtot, &s_total);
  }
  auto walk = [&](auto &&emit) {   // calls emit(b) for every selected block of this thread's range, in order
    int e = eq_rank;
    for (int b = b0; b < b1; ++b) {
      bool sel = mandatory(b);
      if (!sel && Kr > 0) {
        const uint32_t k = keys[b];
        if (ranked) {
          sel = (k & 0x80000000u) != 0 || (k >> 20) > digit0;
        } else if (k > thr) {
          sel = true;
        } else if (k == thr) {
          sel = all_eq || e < need_eq;
          ++e;
        }
      }
      if (sel) emit(b);
    }
  };
  // one pass decides; the thread's selected blocks are remembered as a bit mask (ranges longer than 32 walk twice)
  int c_sel = 0;
  uint32_t picked = 0;
  const bool masked = per <= 32;
  if (ranked && cached && masked) {
    // the usual case in one comparison per key: marked keys carry the sign bit and every key of a higher bin is at
    // least (digit + 1) << 20, so "selected" is an unsigned >= ; mandatory blocks only matter at the two ends
    const uint32_t floor_key = (digit0 + 1u) << 20;
    const bool ends = b0 < P.sink || b1 > X - n_tail;
    for (int b = b0; b < b1; ++b) {
      const bool sel = skeys[b] >= floor_key || (ends && mandatory(b));
      c_sel += sel ? 1 : 0;
      picked |= (sel ? 1u : 0u) << (b - b0);
    }
  } else {
    walk([&](int b) { ++c_sel; if (masked) picked |= 1u << (b - b0); });
  }
  int pos = block_exclusive_scan(c_sel, s_wtot, &s_total);
  const int total = s_total;
  if (masked) {
    while (picked != 0) {
      const int j = __ffs(picked) - 1;
      picked &= picked - 1;
      if (pos < kcap) ids[pos] = b0 + j;
      ++pos;
    }
  } else {
    walk([&](int b) { if (pos < kcap) ids[pos] = b; ++pos; });
  }
  for (int i = total + tid; i < kcap; i += kThreads) ids[i] = -1;
  if (tid == 0) sel_cnt[unit] = min(total, kcap);
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, const int *seq_lens, int units, int kcap, int scan_grid, int *sel_ids, int *sel_cnt,
                     cudaStream_t st) {
  const size_t smem = (size_t)kSmemKeys * sizeof(uint32_t);
  ckv_select_kernel<G><<<units, kThreads, smem, st>>>(c->dev, seq_lens, kcap, scan_grid, units, sel_ids, sel_cnt);
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

cudaError_t ckv_launch_select(ckv_ctx *c, const int *seq_lens, int batch, int kcap, int scan_grid, int *sel_ids,
                              int *sel_cnt, cudaStream_t st) {
  const int units = batch * c->dev.Hkv;
  c->launches++;
  switch (c->dev.G) {
    case 1: return launch_g<1>(c, seq_lens, units, kcap, scan_grid, sel_ids, sel_cnt, st);
    case 2: return launch_g<2>(c, seq_lens, units, kcap, scan_grid, sel_ids, sel_cnt, st);
    case 4: return launch_g<4>(c, seq_lens, units, kcap, scan_grid, sel_ids, sel_cnt, st);
    case 8: return launch_g<8>(c, seq_lens, units, kcap, scan_grid, sel_ids, sel_cnt, st);
  }
  return cudaErrorInvalidValue;
}
