// Summary scan: one streaming pass over every block summary (Eq. 8-9 and the compensation sums
// of Eq. 12), as a persistent, bulk-copy-pipelined kernel.
//
// For every block b and query head g of a unit the pass computes
//   zbar_{g,b}        = q_g . kbar_b * scale                      (block-mean logit, Sec. 4.1)
//   sigma_hat^2_{g,b} = scale^2 sum_t w_{g,t} Dbar_{b,t}         (Eq. 8 with 1/d = scale^2, w_{g,t} = sum_{i in G_t} q_{g,i}^2)
//   l_{g,b}           = log|b| + zbar + sigma_hat^2 / 2           (log of the numerator of Eq. 9)
// and stores (l, sigma_hat^2) for the selection kernel, together with per-CTA partials of the
// normaliser of Eq. 9.  In the same pass it accumulates the mean-compensation terms of Eq. 12 over
// ALL blocks,  sum_b |b| e^{zbar} vbar_b  and  sum_b |b| e^{zbar},  as online-softmax partials; the
// terms of the blocks that end up selected are taken out again by the attention kernel.  That way
// kbar, Dbar and vbar are each read from HBM exactly once per decode step.
//
// Schedule: the summaries of all units are cut into tiles of 32 consecutive blocks; the tiles, in
// (unit, position) order, are split into one contiguous range per CTA and the grid is one CTA per
// SM.  A producer warp streams the CTA's tiles into a ring of shared-memory stages with
// cp.async.bulk (mean-key rows one copy each, so that they land with a padded row stride), completion
// on mbarriers.  Eight consumer warps work on a tile in three phases separated by named barriers:
//   1. mean logits: each thread takes one block (one padded row, conflict-free) and a pair of heads over
//      a slice of the 128 coordinates, the query slice coming from shared memory as a broadcast;
//   2. one thread per (block, head): variance projection, l, the running maximum of the tile, the
//      compensation weight |b| e^{zbar - m}; weights go to shared memory;
//   3. accumulation: a warp takes a mean-value row, each lane four coordinates of all G heads.
// A CTA writes one partial per unit it touched; partial (CTA c, unit u) lives in entry c + u, which
// is unique because the (c, u) pairs that occur form a monotone staircase.
#include "ckv_internal.cuh"
#include "ckv_pipe.cuh"

namespace {

using namespace ckv_pipe;

constexpr int TB = CKV_SCAN_TILE;   // blocks per tile (32: one block per lane in phase 1)
constexpr int KROW = CKV_D + 4;     // padded mean-key row (floats): rows 8 apart share banks, a quarter warp does not
constexpr int kMaxStages = 8;
constexpr int kConsumers = 256;     // 8 consumer warps
constexpr int kThreads = kConsumers + 32;   // plus the producer warp
constexpr int kMaxUnits = 1024;     // sequence lengths are staged in shared memory up to this many sequences

struct UnitInfo { int N, X, tiles; };

__device__ __forceinline__ UnitInfo unit_info(const CkvDev &P, const int *__restrict__ seq_lens, int u) {
  UnitInfo ui;
  ui.N = max(min(seq_lens[u / P.Hkv], P.max_blocks * P.bs), 0);
  ui.X = (ui.N + P.bs - 1) / P.bs;
  ui.tiles = (ui.X + TB - 1) / TB;
  return ui;
}

// Tiles of one sequence's units: from the staged table, or recomputed for sequences beyond it.
__device__ __forceinline__ int seq_tiles(const int *s_tiles, const int *__restrict__ seq_lens, const CkvDev &P, int i) {
  if (i < kMaxUnits) return s_tiles[i];
  const int n = max(min(seq_lens[i], P.max_blocks * P.bs), 0);
  return ((n + P.bs - 1) / P.bs + TB - 1) / TB;
}

// Phase-1 work split: HP heads per thread, the 128 coordinates cut into QD slices, so that the
// (head group, slice) tasks are a multiple of the 8 consumer warps.
template <int G> struct P1Cfg {
  static constexpr int HP = G >= 2 ? 2 : 1;
  static constexpr int HG = G / HP;                       // head groups
  static constexpr int QD = (HG >= 2) ? 4 : 8;            // coordinate slices
  static constexpr int TASKS = HG * QD;                   // warp tasks per tile: 8 (G <= 4) or 16 (G = 8)
  static constexpr int SLICE = CKV_D / QD;                // coordinates per slice
};

template <int G, typename QT>
__global__ void __launch_bounds__(kThreads, 1)
ckv_scan_kernel(CkvDev P, const QT *__restrict__ q, const int *__restrict__ seq_lens, int units, int stages) {
  using C1 = P1Cfg<G>;
  extern __shared__ __align__(128) float stage_mem[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
  __shared__ __align__(16) float sq[G][CKV_D];           // the unit's queries, scaled
  __shared__ __align__(16) float sw[CKV_D][G];           // w_{g,t} * scale^2
  __shared__ __align__(16) float zpart[C1::QD][G][TB];   // phase 1 -> 2: partial mean logits
  __shared__ __align__(16) float2 wbuf[2][TB][G];        // phase 2 -> 3: compensation weights, each stored twice (w, w)
  __shared__ __align__(8) float2 s_scale[2][G];          // phase 2 -> 3: accumulator rescale factors (s, s), 1 unless the
                                                         // running maximum moved; both double-buffered by tile parity
  __shared__ float s_mref[G];                            // flush: the heads' running maxima
  __shared__ __align__(16) float red[G][CKV_D];          // flush: sum of the warps' accumulators
  __shared__ float s_l[8][G], s_lp[8][G];
  __shared__ int s_u0, s_tl0, s_count, s_abort, s_issued, s_consumed;
  __shared__ int s_tiles[kMaxUnits];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool dbar_bulk = P.r >= 4;   // smaller rows cannot keep the 16-byte alignment bulk copies need
  const int stage_floats = TB * KROW + TB * CKV_D + (dbar_bulk ? TB * P.r : 0);

  // tiles per unit from the sequence lengths (staged in shared memory: one parallel load, no serial global reads)
  const int batch = units / P.Hkv;
  for (int i = tid; i < batch && i < kMaxUnits; i += kThreads) {
    const int n = max(min(seq_lens[i], P.max_blocks * P.bs), 0);
    s_tiles[i] = ((n + P.bs - 1) / P.bs + TB - 1) / TB;
  }
  __syncthreads();
  if (tid == 0) {
    long long T = 0;
    for (int i = 0; i < batch; ++i) T += (long long)seq_tiles(s_tiles, seq_lens, P, i) * P.Hkv;
    const long long tpc = (T + gridDim.x - 1) / gridDim.x;
    const long long first = (long long)blockIdx.x * tpc;
    long long cnt = T - first;
    if (cnt > tpc) cnt = tpc;
    if (cnt < 0) cnt = 0;
    int u0 = 0, tl0 = 0;
    if (cnt > 0) {
      long long accum = 0;
      for (int i = 0; i < batch; ++i) {
        const long long t = seq_tiles(s_tiles, seq_lens, P, i);
        if (t > 0 && first < accum + t * P.Hkv) {
          const long long off = first - accum;
          u0 = i * P.Hkv + (int)(off / t); tl0 = (int)(off % t);
          break;
        }
        accum += t * P.Hkv;
      }
    }
    s_u0 = u0; s_tl0 = tl0; s_count = (int)cnt; s_abort = 0; s_issued = 0; s_consumed = 0;
    for (int st = 0; st < stages; ++st) { mbar_init(&full_bar[st], 1); mbar_init(&empty_bar[st], 8); }
    fence_barrier_init();
  }
  __syncthreads();
  const int count = s_count;
  if (count == 0) return;   // uniform: this CTA has no tiles

  if (warp == 8) {
    // ---------------- producer warp: streams the CTA's tiles into the ring ----------------
    int u = s_u0, tl = s_tl0, st = 0;
    uint32_t phase = 0;            // parity of the empty-barrier phase the next refill of stage `st` waits for
    UnitInfo ui = unit_info(P, seq_lens, u);
    for (int it = 0; it < count; ++it) {
      int stop = 0;
      if (lane == 0) {
        if (it >= stages && !mbar_wait(&empty_bar[st], phase)) {
          atomicOr(P.status, CKV_DEV_TIMEOUT);
          *(volatile int *)&s_abort = 1;
        }
        stop = *(volatile int *)&s_abort;
      }
      if (__shfl_sync(0xffffffffu, stop, 0)) break;
      const int b0 = tl * TB;
      const int nb = min(TB, ui.X - b0);
      const size_t row = (size_t)u * P.max_blocks + b0;
      float *sk = stage_mem + (size_t)st * stage_floats;
      float *sv = sk + TB * KROW;
      const uint32_t kbytes = (uint32_t)nb * CKV_D * 4;
      const uint32_t dbytes = dbar_bulk ? (uint32_t)nb * P.r * 4 : 0;
      if (lane == 0) mbar_arrive_expect_tx(&full_bar[st], 2 * kbytes + dbytes);
      __syncwarp();
      if (lane < nb) bulk_g2s(sk + lane * KROW, P.kmean + (row + lane) * CKV_D, CKV_D * 4, &full_bar[st]);
      if (lane == 0) {
        bulk_g2s(sv, P.vmean + row * CKV_D, kbytes, &full_bar[st]);
        if (dbar_bulk) bulk_g2s(sv + TB * CKV_D, P.dbar + row * P.r, dbytes, &full_bar[st]);
        *(volatile int *)&s_issued = it + 1;
      }
      if (++st == stages) { st = 0; if (it >= stages) phase ^= 1; }
      if (++tl == ui.tiles) {
        tl = 0;
        do { ++u; } while (u < units && (ui = unit_info(P, seq_lens, u)).tiles == 0);
      }
    }
  } else {
    // ---------------- consumers ----------------
    // phase 1 role: block = lane; task = (head group, coordinate slice)
    // phase 2 role: one (block, head) per thread; a head's 32 blocks sit in one warp, so its tile maximum is a
    // warp reduction and the (l, sigma^2) stores of the head-major layout coalesce
    const bool p2 = warp < G;              // phase 2: warp g owns head g, lane = block of the tile
    const int p2_bl = lane, p2_g = warp;
    // phase 3 role: rows warp, warp + 8, ...; this lane's four coordinates of all heads
    f32x2 acc[G][2];
    float m_ref = -CUDART_INF_F, l_acc = 0.f, lp_acc = 0.f;   // phase-2 state of head p2_g (same m_ref in every thread of a head)
    float wown[4] = {0.f, 0.f, 0.f, 0.f};
    const bool r4 = P.r == 4 && dbar_bulk;   // the default r: the variance projection is four FMAs on one 16-byte read
    const float log_bs = logf((float)P.bs);
    float log_last = 0.f;
    int u = s_u0, tl = s_tl0, cur = -1, st = 0;
    uint32_t phase = 0;              // parity of the full-barrier phase of stage `st` this pass over the ring
    UnitInfo ui = unit_info(P, seq_lens, u);
    float2 *ls = nullptr;
    const float *db = nullptr;
    bool aborted = false;

    auto flush = [&](int unit_done) {
      // all warps share m_ref, so their accumulators add directly (shared-memory atomics: this runs once per unit)
      for (int idx = tid; idx < G * CKV_D; idx += kConsumers) red[idx / CKV_D][idx % CKV_D] = 0.f;
      named_barrier(1, kConsumers);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float a0, a1, a2, a3;
        unpack2(acc[g][0], a0, a1);
        unpack2(acc[g][1], a2, a3);
        atomicAdd(&red[g][4 * lane], a0); atomicAdd(&red[g][4 * lane + 1], a1);
        atomicAdd(&red[g][4 * lane + 2], a2); atomicAdd(&red[g][4 * lane + 3], a3);
      }
      if (p2) {
        // l and lp of head p2_g: sum over the lanes of its warp
        const float l = warp_sum(l_acc), lp = warp_sum(lp_acc);
        if (lane == 0) { s_l[0][p2_g] = l; s_lp[0][p2_g] = lp; s_mref[p2_g] = m_ref; }
      }
      named_barrier(1, kConsumers);
      float *part = P.comp_part + (size_t)(blockIdx.x + unit_done) * G * CKV_PART_STRIDE;
      for (int idx = tid; idx < G * CKV_D; idx += kConsumers) {
        const int g = idx / CKV_D, i = idx % CKV_D;
        part[g * CKV_PART_STRIDE + 4 + i] = red[g][i];
        if (i == 0) {
          part[g * CKV_PART_STRIDE] = s_mref[g];
          part[g * CKV_PART_STRIDE + 1] = s_l[0][g];
          part[g * CKV_PART_STRIDE + 2] = s_lp[0][g];
        }
      }
      named_barrier(1, kConsumers);
    };

    for (int it = 0; it < count; ++it) {
      if (u != cur) {
        if (cur >= 0) flush(cur);
        // per-unit setup: the unit's queries (scaled), their per-group squared norms, fresh accumulators
        const int s = u / P.Hkv, h = u % P.Hkv;
        for (int idx = tid; idx < G * CKV_D; idx += kConsumers)
          sq[idx / CKV_D][idx % CKV_D] = to_float(q[((size_t)s * P.Hq + h * G) * CKV_D + idx]);
        named_barrier(1, kConsumers);
        for (int idx = tid; idx < P.r * G; idx += kConsumers) {
          const int t = idx / G, g = idx % G;
          float w = 0.f;
          for (int i = 0; i < CKV_D; ++i)
            if (group_of(i, P.r, P.glayout) == t) w = fmaf(sq[g][i], sq[g][i], w);
          sw[t][g] = w * (P.scale * P.scale);   // Eq. 8's 1/d is the squared logit scale
        }
        named_barrier(1, kConsumers);
        for (int idx = tid; idx < G * CKV_D; idx += kConsumers) sq[idx / CKV_D][idx % CKV_D] *= P.scale;
        if (r4 && p2) {
#pragma unroll
          for (int t = 0; t < 4; ++t) wown[t] = sw[t][p2_g];
        }
#pragma unroll
        for (int g = 0; g < G; ++g) { acc[g][0] = pack2(0.f, 0.f); acc[g][1] = pack2(0.f, 0.f); }
        m_ref = -CUDART_INF_F; l_acc = 0.f; lp_acc = 0.f;
        log_last = logf((float)(ui.N - (ui.X - 1) * P.bs));
        const size_t row0 = (size_t)u * P.max_blocks;
        ls = P.ls + row0 * G;   // [head][block] within the unit
        db = P.dbar + row0 * P.r;
        cur = u;
        named_barrier(1, kConsumers);
      }
      // a wait that runs out marks the step invalid; the walk (and its barriers) still runs to the end
      if (!aborted) {
        bool fail = *(volatile int *)&s_abort != 0;
        if (!fail && !mbar_wait(&full_bar[st], phase)) {
          atomicOr(P.status, CKV_DEV_TIMEOUT);
          *(volatile int *)&s_abort = 1;
          fail = true;
        }
        aborted = __any_sync(0xffffffffu, fail);
      }
      const float *sk = stage_mem + (size_t)st * stage_floats;
      const float *sv = sk + TB * KROW;
      const float *sd = sv + TB * CKV_D;
      const int b0 = tl * TB;
      const int nb = min(TB, ui.X - b0);

      // ---- phase 1: partial mean logits, thread = (block lane, head group, coordinate slice) ----
      if (!aborted) {
#pragma unroll
        for (int task = warp; task < C1::TASKS; task += 8) {
          const int hg = task % C1::HG, qd = task / C1::HG;
          const float *krow = sk + lane * KROW + qd * C1::SLICE;
          f32x2 za[C1::HP], zb[C1::HP];
#pragma unroll
          for (int hh = 0; hh < C1::HP; ++hh) { za[hh] = pack2(0.f, 0.f); zb[hh] = pack2(0.f, 0.f); }
#pragma unroll
          for (int c = 0; c < C1::SLICE; c += 4) {
            // 16-byte loads as two packed pairs: no repacking between the load and the packed FMA
            const ulonglong2 k2 = *reinterpret_cast<const ulonglong2 *>(krow + c);
#pragma unroll
            for (int hh = 0; hh < C1::HP; ++hh) {
              const ulonglong2 q2 = *reinterpret_cast<const ulonglong2 *>(&sq[hg * C1::HP + hh][qd * C1::SLICE + c]);
              za[hh] = fma2(q2.x, k2.x, za[hh]);
              zb[hh] = fma2(q2.y, k2.y, zb[hh]);
            }
          }
#pragma unroll
          for (int hh = 0; hh < C1::HP; ++hh) {
            float a0, a1, b0f, b1f;
            unpack2(za[hh], a0, a1);
            unpack2(zb[hh], b0f, b1f);
            zpart[qd][hg * C1::HP + hh][lane] = (a0 + a1) + (b0f + b1f);
          }
        }
      }
      named_barrier(2, kConsumers);

      // ---- phase 2: per (block, head) ----
      float zl2 = -CUDART_INF_F, sig = 0.f;
      bool valid = false;
      if (p2 && !aborted) {
        valid = p2_bl < nb;
        float zbar = 0.f;
#pragma unroll
        for (int qd = 0; qd < C1::QD; ++qd) zbar += zpart[qd][p2_g][p2_bl];
        if (valid) {
          if (r4) {
            const float4 dv = *reinterpret_cast<const float4 *>(sd + p2_bl * 4);
            sig = fmaf(wown[0], dv.x, fmaf(wown[1], dv.y, fmaf(wown[2], dv.z, wown[3] * dv.w)));
          } else {
            for (int t = 0; t < P.r; ++t) {
              const float dv = dbar_bulk ? sd[p2_bl * P.r + t] : __ldg(db + (size_t)(b0 + p2_bl) * P.r + t);
              sig = fmaf(sw[t][p2_g], dv, sig);
            }
          }
          const int b = b0 + p2_bl;
          const float logc = (b == ui.X - 1) ? log_last : log_bs;
          ls[(size_t)p2_g * P.max_blocks + b] = make_float2(logc + zbar + 0.5f * sig, sig);
          zl2 = (zbar + logc) * kLog2e;   // log2 of the compensation weight |b| e^{zbar}
        }
        // the running maximum is only raised when the tile's maximum exceeds it by a slack: weights stay below 2^slack
        const float tm = warp_max(zl2);
        float sc = 1.f;
        if (tm > m_ref + CKV_RESCALE_SLACK) {
          sc = exp2_diff(m_ref, tm);
          m_ref = tm;
          l_acc *= sc; lp_acc *= sc;
        }
        if (lane == 0) s_scale[it & 1][p2_g] = make_float2(sc, sc);
        const float wt = valid ? fast_exp2(zl2 - m_ref) : 0.f;
        wbuf[it & 1][p2_bl][p2_g] = make_float2(wt, wt);
        l_acc += wt;
        lp_acc = fmaf(wt, fast_exp2(0.5f * kLog2e * sig), lp_acc);   // e^{l - m} = e^{zbar + log|b| - m} e^{sigma^2/2}
      }
      named_barrier(2, kConsumers);

      // ---- phase 3: acc_g += w_{g,b} vbar_b, a warp per row, four coordinates per lane ----
      if (!aborted) {
        const f32x2 *scp = reinterpret_cast<const f32x2 *>(s_scale[it & 1]);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const f32x2 sc2 = scp[g];
          acc[g][0] = mul2(acc[g][0], sc2);
          acc[g][1] = mul2(acc[g][1], sc2);
        }
#pragma unroll
        for (int j = 0; j < TB / 8; ++j) {
          const int bl = warp + 8 * j;
          if (bl < nb) {   // rows past the unit's last block hold stale bytes
            const ulonglong2 v2 = *reinterpret_cast<const ulonglong2 *>(sv + bl * CKV_D + 4 * lane);
            const f32x2 *wp = reinterpret_cast<const f32x2 *>(wbuf[it & 1][bl]);
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const f32x2 w2 = wp[g];
              acc[g][0] = fma2(w2, v2.x, acc[g][0]);
              acc[g][1] = fma2(w2, v2.y, acc[g][1]);
            }
          }
        }
      }
      // the stage is free once every warp has read its rows (the weights are double-buffered, so the next
      // tile's phase 2 may start while slower warps are still here)
      __syncwarp();
      if (lane == 0 && !aborted) {
        mbar_arrive(&empty_bar[st]);
        if (warp == 0) *(volatile int *)&s_consumed = it + 1;
      }
      if (++st == stages) { st = 0; phase ^= 1; }
      if (++tl == ui.tiles) {
        tl = 0;
        do { ++u; } while (u < units && (ui = unit_info(P, seq_lens, u)).tiles == 0);
      }
    }
    if (cur >= 0) flush(cur);
  }
  __syncthreads();
  if (s_abort && tid == 0) {
    // leave no bulk copy in flight into this CTA's shared memory: wait (bounded) for every issued fill
    for (int it = s_consumed; it < s_issued; ++it) mbar_wait(&full_bar[it % stages], (it / stages) & 1);
  }
}

struct ScanCfg { int stages; size_t smem; };

template <int G>
ScanCfg scan_cfg(const CkvDev &P) {
  using C1 = P1Cfg<G>;
  const size_t stage_bytes = ((size_t)TB * KROW + (size_t)TB * CKV_D + (P.r >= 4 ? (size_t)TB * P.r : 0)) * 4;
  const size_t fixed = (size_t)G * CKV_D * 4 + (size_t)CKV_D * G * 4 + (size_t)C1::QD * TB * G * 4 + (size_t)TB * G * 4 +
                       (size_t)G * CKV_D * 4 + (size_t)kMaxUnits * 4 + 2048;
  const size_t budget = 224 * 1024 - fixed;
  int stages = (int)(budget / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) stages = 2;
  return ScanCfg{stages, stages * stage_bytes};
}

template <int G, typename QT>
cudaError_t launch_gt(ckv_ctx *c, const void *q, const int *seq_lens, int units, int grid, cudaStream_t st) {
  const ScanCfg cfg = scan_cfg<G>(c->dev);
  ckv_scan_kernel<G, QT><<<grid, kThreads, cfg.smem, st>>>(c->dev, (const QT *)q, seq_lens, units, cfg.stages);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, const void *q, const int *seq_lens, int units, int grid, cudaStream_t st) {
  if (c->layout.kv_dtype == CKV_BF16) return launch_gt<G, __nv_bfloat16>(c, q, seq_lens, units, grid, st);
  return launch_gt<G, float>(c, q, seq_lens, units, grid, st);
}

template <int G, typename QT>
cudaError_t configure_gt(const ckv_ctx *c) {
  return cudaFuncSetAttribute(ckv_scan_kernel<G, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)scan_cfg<G>(c->dev).smem);
}

template <int G>
cudaError_t configure_g(const ckv_ctx *c) {
  if (c->layout.kv_dtype == CKV_BF16) return configure_gt<G, __nv_bfloat16>(c);
  return configure_gt<G, float>(c);
}

}  // namespace

// Opt in to the dynamic shared memory this context's scan instantiation needs, on the current device.
cudaError_t ckv_configure_scan(const ckv_ctx *c) {
  switch (c->dev.G) {
    case 1: return configure_g<1>(c);
    case 2: return configure_g<2>(c);
    case 4: return configure_g<4>(c);
    case 8: return configure_g<8>(c);
  }
  return cudaErrorInvalidValue;
}

// Grid size the scan uses for a step (one persistent CTA per SM, never more CTAs than tiles).
int ckv_scan_grid(const ckv_ctx *c, int batch, int max_len) {
  const CkvDev &P = c->dev;
  const int xmax = (max_len + P.bs - 1) / P.bs;
  const long long tiles = (long long)batch * P.Hkv * ((xmax + TB - 1) / TB);
  long long grid = c->sm_count;
  if (grid > CKV_MAX_SCAN_CTAS) grid = CKV_MAX_SCAN_CTAS;
  if (grid > tiles) grid = tiles;
  return (int)(grid < 1 ? 1 : grid);
}

cudaError_t ckv_launch_scan(ckv_ctx *c, const void *q, const int *seq_lens, int batch, int max_len, int *grid_out,
                            cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int units = batch * P.Hkv;
  const int grid = ckv_scan_grid(c, batch, max_len);
  *grid_out = grid;
  c->launches++;
  switch (P.G) {
    case 1: return launch_g<1>(c, q, seq_lens, units, grid, st);
    case 2: return launch_g<2>(c, q, seq_lens, units, grid, st);
    case 4: return launch_g<4>(c, q, seq_lens, units, grid, st);
    case 8: return launch_g<8>(c, q, seq_lens, units, grid, st);
  }
  return cudaErrorInvalidValue;
}
