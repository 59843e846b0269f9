// Summary scan: one streaming pass over every block summary (Eq. 8-9 and the compensation sums
// of Eq. 12), as a persistent, bulk-copy-pipelined kernel.
//
// For every block b and query head g of a unit the pass computes
//   zbar_{g,b}        = q_g . kbar_b * scale                      (block-mean logit, Sec. 4.1)
//   sigma_hat^2_{g,b} = scale^2 sum_t w_{g,t} Dbar_{b,t}         (Eq. 8 with 1/d = scale^2, w_{g,t} = sum_{i in G_t} q_{g,i}^2)
//   l_{g,b}           = log|b| + zbar + sigma_hat^2 / 2           (log of the numerator of Eq. 9)
// and stores (l, sigma_hat^2) for the selection kernel.  In the same pass it accumulates the
// mean-compensation terms of Eq. 12 over ALL blocks,  sum_b |b| e^{zbar} vbar_b  and
// sum_b |b| e^{zbar},  as online-softmax partials; the terms of the blocks that end up selected
// are taken out again by the attention kernel.  That way kbar, Dbar and vbar are each read
// from HBM exactly once per decode step.
//
// Schedule: the summaries of all units are cut into tiles of 16 consecutive blocks (16 KB of mean
// keys + 16 KB of mean values + the variances); the tiles, in (unit, position) order, are split
// into one contiguous range per CTA and the grid is one CTA per SM.  A producer thread streams the
// CTA's tiles into a ring of shared-memory stages with cp.async.bulk, completion on mbarriers;
// eight consumer warps take two blocks each per tile.  A CTA writes one partial per unit it
// touched; partial (CTA c, unit u) lives in entry c + u, which is unique because the (c, u)
// pairs that occur form a monotone staircase.
//
// Consumer mapping: 16 lanes share one block row (128 fp32 = 32 float4; lane li takes float4 li and
// li + 16, conflict-free in shared memory); each lane keeps its 8 coordinates of q (all G heads) and
// of the G output accumulators in registers.
#include "ckv_internal.cuh"
#include "ckv_pipe.cuh"

namespace {

using namespace ckv_pipe;

template <int G> struct Log2 { static constexpr int v = 1 + Log2<G / 2>::v; };
template <> struct Log2<1> { static constexpr int v = 0; };

constexpr int TB = CKV_SCAN_TILE;   // blocks per tile
constexpr int kMaxStages = 8;
constexpr int NP = TB / 16;          // row pairs a consumer warp takes per tile
constexpr int kConsumers = 256;     // 8 consumer warps
constexpr int kThreads = kConsumers + 32;   // plus one producer warp (a single thread of it issues the bulk copies)
constexpr int kMaxUnits = 1024;     // sequence lengths are staged in shared memory up to this many sequences

struct UnitInfo { int N, X, tiles; };

// Tiles of one sequence's units: from the staged table, or recomputed for sequences beyond it.
__device__ __forceinline__ int seq_tiles(const int *s_tiles, const int *__restrict__ seq_lens, const CkvDev &P, int i) {
  if (i < kMaxUnits) return s_tiles[i];
  const int n = max(min(seq_lens[i], P.max_blocks * P.bs), 0);
  return ((n + P.bs - 1) / P.bs + TB - 1) / TB;
}

__device__ __forceinline__ UnitInfo unit_info(const CkvDev &P, const int *__restrict__ seq_lens, int u) {
  UnitInfo ui;
  ui.N = min(seq_lens[u / P.Hkv], P.max_blocks * P.bs);
  ui.N = max(ui.N, 0);
  ui.X = (ui.N + P.bs - 1) / P.bs;
  ui.tiles = (ui.X + TB - 1) / TB;
  return ui;
}

template <int G, typename QT>
__global__ void __launch_bounds__(kThreads, 1)
ckv_scan_kernel(CkvDev P, const QT *__restrict__ q, const int *__restrict__ seq_lens, int units, int stages) {
  constexpr int SH = 4 - Log2<G>::v;   // lane (g << SH) of a half warp owns head g after the reduction
  extern __shared__ __align__(128) float stage_mem[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
  __shared__ float sq[G][CKV_D];
  __shared__ __align__(16) float sw[CKV_D][G];
  __shared__ __align__(16) float red[8][G][CKV_PART_STRIDE];
  __shared__ int s_u0, s_tl0, s_count, s_abort, s_issued, s_consumed;
  __shared__ int s_tiles[kMaxUnits];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 4, li = lane & 15;
  const bool dbar_bulk = P.r >= 4;   // smaller rows cannot keep the 16-byte alignment bulk copies need
  const int stage_floats = TB * 2 * CKV_D + (dbar_bulk ? TB * P.r : 0);

  // tiles per unit from the sequence lengths (staged in shared memory: one parallel load, no serial global reads)
  const int batch = units / P.Hkv;
  for (int i = tid; i < batch && i < kMaxUnits; i += kThreads) {
    const int n = max(min(seq_lens[i], P.max_blocks * P.bs), 0);
    s_tiles[i] = ((n + P.bs - 1) / P.bs + TB - 1) / TB;
  }
  __syncthreads();
  if (tid == 0) {
    long long T = 0;
    for (int sq_i = 0; sq_i < batch; ++sq_i) T += (long long)seq_tiles(s_tiles, seq_lens, P, sq_i) * P.Hkv;
    const long long tpc = (T + gridDim.x - 1) / gridDim.x;
    const long long first = (long long)blockIdx.x * tpc;
    long long cnt = T - first;
    if (cnt > tpc) cnt = tpc;
    if (cnt < 0) cnt = 0;
    int u0 = 0, tl0 = 0;
    if (cnt > 0) {
      long long accum = 0;
      for (int sq_i = 0; sq_i < batch; ++sq_i) {
        const long long t = seq_tiles(s_tiles, seq_lens, P, sq_i);
        if (t > 0 && first < accum + t * P.Hkv) {
          const long long off = first - accum;
          u0 = sq_i * P.Hkv + (int)(off / t); tl0 = (int)(off % t);
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
    // ---------------- producer: one thread streams the CTA's tiles into the ring ----------------
    if (lane == 0) {
      int u = s_u0, tl = s_tl0, st = 0;
      uint32_t phase = 0;            // parity of the empty-barrier phase the next refill of stage `st` waits for
      UnitInfo ui = unit_info(P, seq_lens, u);
      for (int it = 0; it < count; ++it) {
        if (it >= stages && !mbar_wait(&empty_bar[st], phase)) {
          atomicOr(P.status, CKV_DEV_TIMEOUT);
          *(volatile int *)&s_abort = 1;
        }
        if (*(volatile int *)&s_abort) break;
        const int b0 = tl * TB;
        const int nb = min(TB, ui.X - b0);
        const size_t row = (size_t)u * P.max_blocks + b0;
        float *sk = stage_mem + (size_t)st * stage_floats;
        float *sv = sk + TB * CKV_D;
        const uint32_t kbytes = (uint32_t)nb * CKV_D * 4;
        const uint32_t dbytes = dbar_bulk ? (uint32_t)nb * P.r * 4 : 0;
        mbar_arrive_expect_tx(&full_bar[st], 2 * kbytes + dbytes);
        bulk_g2s(sk, P.kmean + row * CKV_D, kbytes, &full_bar[st]);
        bulk_g2s(sv, P.vmean + row * CKV_D, kbytes, &full_bar[st]);
        if (dbar_bulk) bulk_g2s(sv + TB * CKV_D, P.dbar + row * P.r, dbytes, &full_bar[st]);
        *(volatile int *)&s_issued = it + 1;
        if (++st == stages) { st = 0; if (it >= stages) phase ^= 1; }
        if (++tl == ui.tiles) {
          tl = 0;
          do { ++u; } while (u < units && (ui = unit_info(P, seq_lens, u)).tiles == 0);
        }
      }
    }
  } else {
    // ---------------- consumers ----------------
    f32x2 qr[G][4], acc[G][4];   // this lane's 8 coordinates (4 pairs) of every head's query and accumulator
    float m_ref[G], wown[4];
    float m_my = -CUDART_INF_F, l_my = 0.f, lp_my = 0.f;   // lp: sum of e^{l - m}, the normaliser of Eq. 9
    const bool r4 = P.r == 4 && dbar_bulk;   // the default r: the owner lane evaluates Eq. 8 by itself
    const int myg = li >> SH;
    const float log_bs = logf((float)P.bs);
    float log_last = 0.f;
    int u = s_u0, tl = s_tl0, cur = -1, st = 0;
    uint32_t phase = 0;              // parity of the full-barrier phase of stage `st` this pass over the ring
    UnitInfo ui = unit_info(P, seq_lens, u);
    float2 *ls = nullptr;
    const float *db = nullptr;
    bool aborted = false;

    auto flush = [&](int unit_done) {
      // fold the two half warps, then the 8 warps, into one partial per head of `unit_done`
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float mo = __shfl_xor_sync(0xffffffffu, m_ref[g], 16);
        const float mn = fmaxf(m_ref[g], mo);
        const float sc = exp2_diff(m_ref[g], mn);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float a0, a1;
          unpack2(acc[g][i], a0, a1);
          a0 *= sc; a1 *= sc;
          a0 += __shfl_xor_sync(0xffffffffu, a0, 16);
          a1 += __shfl_xor_sync(0xffffffffu, a1, 16);
          acc[g][i] = pack2(a0, a1);
        }
        float lg = (myg == g) ? l_my * sc : 0.f;
        float lpg = (myg == g) ? lp_my * sc : 0.f;
        lg += __shfl_xor_sync(0xffffffffu, lg, 16);
        lpg += __shfl_xor_sync(0xffffffffu, lpg, 16);
        if (myg == g) { l_my = lg; lp_my = lpg; }
        m_ref[g] = mn;
      }
      if (gid == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float *r = red[warp][g];
          float a[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) unpack2(acc[g][i], a[2 * i], a[2 * i + 1]);
          *reinterpret_cast<float4 *>(r + 4 + 4 * li) = make_float4(a[0], a[1], a[2], a[3]);
          *reinterpret_cast<float4 *>(r + 4 + 64 + 4 * li) = make_float4(a[4], a[5], a[6], a[7]);
          if (li == (g << SH)) { r[0] = m_ref[g]; r[1] = l_my; r[2] = lp_my; }
        }
      }
      named_barrier(1, kConsumers);
      float *part = P.comp_part + (size_t)(blockIdx.x + unit_done) * G * CKV_PART_STRIDE;
      for (int idx = tid; idx < G * CKV_D; idx += kConsumers) {
        const int g = idx / CKV_D, i = idx % CKV_D;
        float M = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < 8; ++w) M = fmaxf(M, red[w][g][0]);
        float num = 0.f, den = 0.f, denp = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const float sc = exp2_diff(red[w][g][0], M);
          num = fmaf(red[w][g][4 + i], sc, num);
          den = fmaf(red[w][g][1], sc, den);
          denp = fmaf(red[w][g][2], sc, denp);
        }
        part[g * CKV_PART_STRIDE + 4 + i] = num;
        if (i == 0) {
          part[g * CKV_PART_STRIDE] = M; part[g * CKV_PART_STRIDE + 1] = den; part[g * CKV_PART_STRIDE + 2] = denp;
        }
      }
      named_barrier(1, kConsumers);
    };

    for (int it = 0; it < count; ++it) {
      if (u != cur) {
        if (cur >= 0) flush(cur);
        // per-unit setup: the unit's queries, their per-group squared norms, fresh accumulators
        const int s = u / P.Hkv, h = u % P.Hkv;
        for (int idx = tid; idx < G * CKV_D; idx += kConsumers)
          sq[idx / CKV_D][idx % CKV_D] = to_float(q[((size_t)s * P.Hq + h * G) * CKV_D + idx]);
        named_barrier(1, kConsumers);
        for (int idx = tid; idx < P.r * G; idx += kConsumers) {
          const int t = idx / G, g = idx % G;
          float w = 0.f;
          for (int i = 0; i < CKV_D; ++i)
            if (group_of(i, P.r, P.glayout) == t) w = fmaf(sq[g][i], sq[g][i], w);
          sw[t][g] = w;
        }
        named_barrier(1, kConsumers);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          m_ref[g] = -CUDART_INF_F;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            qr[g][i] = pack2(sq[g][4 * li + 2 * i] * P.scale, sq[g][4 * li + 2 * i + 1] * P.scale);
            qr[g][2 + i] = pack2(sq[g][64 + 4 * li + 2 * i] * P.scale, sq[g][64 + 4 * li + 2 * i + 1] * P.scale);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[g][i] = pack2(0.f, 0.f);
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) wown[t] = r4 ? sw[t][myg] * (P.scale * P.scale) : 0.f;
        m_my = -CUDART_INF_F; l_my = 0.f; lp_my = 0.f;
        log_last = logf((float)(ui.N - (ui.X - 1) * P.bs));
        const size_t row0 = (size_t)u * P.max_blocks;
        ls = P.ls + row0 * G;
        db = P.dbar + row0 * P.r;
        cur = u;
      }
      // a wait that runs out marks the step invalid; the walk (and its barriers) still runs to the end
      if (!aborted && *(volatile int *)&s_abort) aborted = true;
      if (!aborted && !mbar_wait(&full_bar[st], phase)) {
        atomicOr(P.status, CKV_DEV_TIMEOUT);
        *(volatile int *)&s_abort = 1;
        aborted = true;
      }
      aborted = __any_sync(0xffffffffu, aborted);
      if (aborted) {
        if (++st == stages) { st = 0; phase ^= 1; }
        if (++tl == ui.tiles) {
          tl = 0;
          do { ++u; } while (u < units && (ui = unit_info(P, seq_lens, u)).tiles == 0);
        }
        continue;
      }
      const float *sk = stage_mem + (size_t)st * stage_floats;
      const float *sv = sk + TB * CKV_D;
      const float *sd = sv + TB * CKV_D;
      const int b0 = tl * TB;
      const int nb = min(TB, ui.X - b0);
      // this warp's NP row pairs of the tile: rows warp * 2 NP + 2 p + gid; the pairs are independent
      // chains the compiler interleaves
      int bl[NP];
      bool valid[NP];
      f32x2 kk[NP][4], vv[NP][4];
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        bl[p] = warp * (2 * NP) + 2 * p + gid;
        valid[p] = bl[p] < nb;
        const float4 k0 = *reinterpret_cast<const float4 *>(sk + bl[p] * CKV_D + 4 * li);
        const float4 k1 = *reinterpret_cast<const float4 *>(sk + bl[p] * CKV_D + 64 + 4 * li);
        const float4 v0 = *reinterpret_cast<const float4 *>(sv + bl[p] * CKV_D + 4 * li);
        const float4 v1 = *reinterpret_cast<const float4 *>(sv + bl[p] * CKV_D + 64 + 4 * li);
        kk[p][0] = pack2(k0.x, k0.y); kk[p][1] = pack2(k0.z, k0.w); kk[p][2] = pack2(k1.x, k1.y); kk[p][3] = pack2(k1.z, k1.w);
        vv[p][0] = pack2(v0.x, v0.y); vv[p][1] = pack2(v0.z, v0.w); vv[p][2] = pack2(v1.x, v1.y); vv[p][3] = pack2(v1.z, v1.w);
        if (nb < TB && !valid[p]) {   // rows past the unit's last block hold stale bytes
#pragma unroll
          for (int i = 0; i < 4; ++i) { kk[p][i] = pack2(0.f, 0.f); vv[p][i] = pack2(0.f, 0.f); }
        }
      }
      float zbar[NP], sig[NP];
      if (r4) {
        // r = 4: reduce the G mean logits only; the owner lane of a head evaluates sigma_hat^2 from the
        // block's four group variances (one 16-byte read) with its head's weights held in registers
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          float zr[G];
#pragma unroll
          for (int g = 0; g < G; ++g) {
            f32x2 z2 = mul2(qr[g][0], kk[p][0]);
#pragma unroll
            for (int i = 1; i < 4; ++i) z2 = fma2(qr[g][i], kk[p][i], z2);
            float z0, z1;
            unpack2(z2, z0, z1);
            zr[g] = z0 + z1;
          }
          reduce16<G, 1>(zr, li);
          const float4 dv = *reinterpret_cast<const float4 *>(sd + bl[p] * 4);
          zbar[p] = zr[0];
          sig[p] = fmaf(wown[0], dv.x, fmaf(wown[1], dv.y, fmaf(wown[2], dv.z, wown[3] * dv.w)));
        }
      } else {
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          float red_v[2 * G];
#pragma unroll
          for (int g = 0; g < G; ++g) red_v[2 * g + 1] = 0.f;
          if (valid[p]) {
            for (int t = li; t < P.r; t += 16) {
              const float dv = dbar_bulk ? sd[bl[p] * P.r + t] : __ldg(db + (size_t)(b0 + bl[p]) * P.r + t);
#pragma unroll
              for (int g = 0; g < G; ++g) red_v[2 * g + 1] = fmaf(sw[t][g], dv, red_v[2 * g + 1]);
            }
          }
#pragma unroll
          for (int g = 0; g < G; ++g) {
            f32x2 z2 = mul2(qr[g][0], kk[p][0]);
#pragma unroll
            for (int i = 1; i < 4; ++i) z2 = fma2(qr[g][i], kk[p][i], z2);
            float z0, z1;
            unpack2(z2, z0, z1);
            red_v[2 * g] = z0 + z1;
          }
          reduce16<2 * G, 2>(red_v, li);
          zbar[p] = red_v[0];
          sig[p] = red_v[1] * (P.scale * P.scale);   // Eq. 8's 1/d is the squared logit scale
        }
      }
      float zl2[NP];
      bool raise = false;
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        const int b = b0 + bl[p];
        const float logc = (b == ui.X - 1) ? log_last : log_bs;
        const float ell = logc + zbar[p] + 0.5f * sig[p];
        if (valid[p] && (li & ((1 << SH) - 1)) == 0) ls[(size_t)b * G + myg] = make_float2(ell, sig[p]);
        // compensation weight of this block for head myg: |b| e^{zbar}, in log2 units
        zl2[p] = valid[p] ? (zbar[p] + logc) * kLog2e : -CUDART_INF_F;
        raise |= zl2[p] > m_my + CKV_RESCALE_SLACK;
      }
      if (__any_sync(0xffffffffu, raise)) {
#pragma unroll
        for (int p = 0; p < NP; ++p) {
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float cand = __shfl_sync(0xffffffffu, zl2[p], (lane & 16) | (g << SH));
            if (cand > m_ref[g]) {
              const float sc = exp2_diff(m_ref[g], cand);
              const f32x2 sc2 = pack2(sc, sc);
#pragma unroll
              for (int i = 0; i < 4; ++i) acc[g][i] = mul2(acc[g][i], sc2);
              if (myg == g) { l_my *= sc; lp_my *= sc; m_my = cand; }
              m_ref[g] = cand;
            }
          }
        }
      }
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        // rows past the end contribute nothing (their shared-memory bytes are stale, and m_my may still be -inf)
        const float wt = valid[p] ? fast_exp2(zl2[p] - m_my) : 0.f;
        l_my += wt;
        if (valid[p]) lp_my = fmaf(wt, fast_exp2(0.5f * kLog2e * sig[p]), lp_my);   // e^{l - m} = e^{zbar + log|b| - m} e^{sigma^2/2}
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float wg = __shfl_sync(0xffffffffu, wt, (lane & 16) | (g << SH));
          const f32x2 w2 = pack2(wg, wg);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[g][i] = fma2(w2, vv[p][i], acc[g][i]);
        }
      }
      __syncwarp();
      if (lane == 0) {
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

ScanCfg scan_cfg(const CkvDev &P, int G) {
  const size_t stage_bytes = (size_t)TB * 2 * CKV_D * 4 + (P.r >= 4 ? (size_t)TB * P.r * 4 : 0);
  const size_t fixed = (size_t)G * CKV_D * 4 + (size_t)CKV_D * G * 4 + (size_t)8 * G * CKV_PART_STRIDE * 4 + 1024;
  const size_t budget = 220 * 1024 - fixed;
  int stages = (int)(budget / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) stages = 2;
  return ScanCfg{stages, stages * stage_bytes};
}

template <int G, typename QT>
cudaError_t launch_gt(ckv_ctx *c, const void *q, const int *seq_lens, int units, int grid, cudaStream_t st) {
  const ScanCfg cfg = scan_cfg(c->dev, G);
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
                              (int)scan_cfg(c->dev, G).smem);
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
