// Summary scan: one streaming pass over every block summary (Eq. 8-9 and the compensation sums
// of Eq. 12), as a persistent, bulk-copy-pipelined, tensor-core kernel.
//
// For every block b and query head g of a unit the pass computes
//   zbar_{g,b}        = q_g . kbar_b * scale                      (block-mean logit, Sec. 4.1)
//   sigma_hat^2_{g,b} = scale^2 sum_t w_{g,t} Dbar_{b,t}         (Eq. 8 with 1/d = scale^2, w_{g,t} = sum_{i in G_t} q_{g,i}^2)
//   l_{g,b}           = log|b| + zbar + sigma_hat^2 / 2           (log of the numerator of Eq. 9)
// and stores, in log2 units, e^l sigma_hat^2 for the selection kernel and |b| e^{zbar} for the attention kernel
// (4 bytes each per head and block), together with partials of the normaliser of Eq. 9.  In the same pass it accumulates the mean-compensation terms of Eq. 12 over ALL blocks,
// sum_b |b| e^{zbar} vbar_b  and  sum_b |b| e^{zbar},  as online-softmax partials; the terms of the
// blocks that end up selected are taken out again by the attention kernel.  That way kbar, Dbar and
// vbar are each read from HBM exactly once per decode step.
//
// The two contractions are the GQA-grouped Q Kbar^T and W Vbar tiles, on mma.sync.m16n8k16 (bf16 in,
// fp32 accumulate): heads are the M dimension (G <= 8 rows of 16 used), 8 blocks the N dimension of
// Q Kbar^T, whose accumulator layout is the A-operand layout of W Vbar.  The summaries are stored as
// split bf16 pairs (hi + lo), so x * y is hi * y + lo * y with no conversion instructions; the weights
// w = |b| e^{zbar - m} are split the same way (three products per tile: hi hi, lo hi, hi lo).
//
// Schedule: the launch has two kinds of CTAs.  The first few ("tail" CTAs, one warp per unit) take the LAST block
// of every sequence -- the only block a decode step can change -- and, in a fused step, first append the step's new
// token to it (page write + block summary); see scan_tail.  All other blocks of all units are cut into tiles of
// 32 consecutive blocks; the tiles, in (unit, position) order, are split into one contiguous range per scan CTA,
// one scan CTA per remaining SM.  A producer thread streams the CTA's tiles into a ring of shared-memory stages
// with cp.async.bulk (two 16 KB copies and the variances per tile), completion on mbarriers.  Each of the seven
// consumer warps takes every seventh half tile (16 blocks) on its own and visits only the tiles that hold one of
// its parts -- there is no CTA-wide barrier in the loop -- with a per-warp running maximum that is only raised
// when exceeded by a slack.  The query rows and variance weights of the CTA's units are staged in shared memory
// while the first fills are in flight, so a warp that moves on to another unit sets up from there.  A warp writes one
// partial per unit its CTA touched; partial (scan CTA c, warp w, unit u) lives in entry (c + 2 u) * 7 + w, unique
// because the (c, u) pairs that occur form a monotone staircase; the entry behind a unit's last one is free and
// takes the last block's partial, so a unit's partials are one contiguous run (unit_scan_entries).
//
// Lengths in a fused step: every CTA reads the lengths as they were before the append and works with them plus
// one; a counter of CTAs that are done reading decides who stores the new lengths (lens_arrive), so the kernels
// that follow in the stream see them in place and nobody waits on anybody inside the launch.
#include <algorithm>
#include <mutex>

#include "ckv_internal.cuh"
#include "ckv_pipe.cuh"
#include "ckv_mma.cuh"
#include "ckv_blockstats.cuh"

namespace {

using namespace ckv_pipe;

template <bool WIDE> struct ScanTile { static constexpr int TB = WIDE ? CKV_SCAN_TILE_HS : CKV_SCAN_TILE; };   // blocks per tile

// One box of a tensor map from global to shared memory (x: first element of the row, y: first row); completion is
// counted on `bar` in bytes -- always the whole box, rows past the tensor's end arriving as zeros.
__device__ __forceinline__ void tensor_g2s(uint32_t dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(ckv_pipe::smem_u32(bar))
               : "memory");
}
constexpr int kMaxStages = 8;
constexpr int kConsumerWarps = CKV_SCAN_WARPS;
constexpr int kThreads = kConsumerWarps * 32 + 32;   // plus the producer warp
constexpr int kMaxSeqs = 1024;      // sequence lengths are staged in shared memory up to this many sequences

struct UnitInfo { int N, X, tiles; };   // X: the blocks the scan CTAs cover (in tail mode all but the sequence's last one)

// s_len holds the clamped lengths (after this step's append, if any) of the first kMaxSeqs sequences, staged once
// per CTA; longer batches never come with an append and read the device array
__device__ __forceinline__ int seq_len_of(const CkvDev &P, const int *s_len, const int *__restrict__ seq_lens, int s) {
  return s < kMaxSeqs ? s_len[s] : max(min(seq_lens[s], P.max_blocks * P.bs), 0);
}
__device__ __forceinline__ UnitInfo unit_info(const CkvDev &P, const int *s_len, const int *__restrict__ seq_lens, int u) {
  UnitInfo ui;
  ui.N = seq_len_of(P, s_len, seq_lens, ckv_div_hkv(P, u));
  ui.X = ckv_scan_blocks(P, ui.N);
  ui.tiles = (ui.X + P.scan_tile - 1) >> P.lg_tile;
  return ui;
}

__device__ __forceinline__ int seq_tiles(const int *s_len, const int *__restrict__ seq_lens, const CkvDev &P, int i) {
  return (ckv_scan_blocks(P, seq_len_of(P, s_len, seq_lens, i)) + P.scan_tile - 1) >> P.lg_tile;
}

constexpr int kLenCounter = 16;   // word of the status region that counts the CTAs which have read the lengths

// Length hand-over of a fused step.  Every CTA of the launch works with the lengths as they were before the
// append (plus one); a CTA calls this once it will not read the length array again, and the last one to call
// stores the new lengths, so that the kernels that follow find them in place.  Nobody waits: it is a counter.
// whole_cta: called by all threads of the CTA (which then share the stores), else by one thread.
__device__ __noinline__ void lens_arrive(int *counter, const int *seq_lens, int *seq_lens_out, int batch, int cap,
                                         int n_ctas, bool whole_cta) {
  if (whole_cta) {
    __shared__ int s_is_last;
    __syncthreads();
    if (threadIdx.x == 0) {
      s_is_last = atomicAdd(counter, 1) == n_ctas - 1;
      if (s_is_last) *counter = 0;   // ready for the next launch
    }
    __syncthreads();
    if (!s_is_last) return;
    for (int i = threadIdx.x; i < batch; i += blockDim.x) {
      const int raw = seq_lens[i];
      if (raw >= 0 && raw < cap) seq_lens_out[i] = raw + 1;
    }
  } else {
    if (atomicAdd(counter, 1) != n_ctas - 1) return;
    *counter = 0;
    for (int i0 = 0; i0 < batch; i0 += 8) {   // loads of a group first: the arrays are one and the same
      int raw[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) raw[k] = i0 + k < batch ? seq_lens[i0 + k] : -1;
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (raw[k] >= 0 && raw[k] < cap) seq_lens_out[i0 + k] = raw[k] + 1;
    }
  }
}

// Tail CTAs of the scan launch: one warp per unit.  With a new token (fused step) the warp first stores the
// token's key and value rows into their page and recomputes the summary of the block they land in, with the
// routine the stand-alone append uses.  Then, new token or not, it does for the unit's LAST block what the scan
// CTAs do for all the others -- the block's two per-head terms and its mean-compensation partial -- reading the
// summary as stored.  The last block is the only one a step can change, so the scan CTAs depend on nothing this
// warp writes and the append costs the step no time of its own.
//
// Deliberately not inlined, and with the kernel's parameter block passed BY VALUE: inlined, its code doubled the
// kernel's size and the scan CTAs stalled on instruction fetch (the launch went from 55 to 68 us); handed a
// reference, the compiler moves the parameter block to local memory for every CTA, scan loop included.
template <int G, typename QT>
__device__ __noinline__ void scan_tail(const CkvDev P, const QT *__restrict__ q, const int *seq_lens, int *s_len,
                                       int len_mine, int units, int nscan, const CkvNewToken fresh, int n_tail,
                                       float *smem_f, int smem_bytes) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, hw = lane >> 4, li = lane & 15;
  const int batch = ckv_div_hkv(P, units), cap = P.max_blocks * P.bs;
  const bool append = fresh.k_new != nullptr;
  const bool lo_half = P.row_elems == CKV_ROW_ELEMS;
  const bool by_mass = (P.variant & CKV_VARIANT_RANK_BY_MASS) != 0;
  QT *k_pool = reinterpret_cast<QT *>(fresh.k_pool), *v_pool = reinterpret_cast<QT *>(fresh.v_pool);
  const QT *k_new = reinterpret_cast<const QT *>(fresh.k_new), *v_new = reinterpret_cast<const QT *>(fresh.v_new);
  float *sq = smem_f + warp * CKV_D;
  constexpr int PIECES = (int)(CKV_D * sizeof(QT) / 16);   // 16-byte pieces of a row: lanes 0-15 hold K, 16-31 hold V
  constexpr int PP = PIECES / 16;
  const int u_first = (int)blockIdx.x * 8 + warp;
  // the new row of the warp's first unit does not depend on the lengths: it is requested together with them
  uint4 piece[PP];
  // the unit's G query rows are read head by head in a rolled loop further down (this routine's time is the fetch
  // of its own instructions, executed once per launch: a short loop beats unrolled code); the L2 is asked for them
  // now, while nothing depends on them
  if (u_first < units && lane < G)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(q + ((size_t)u_first * G + lane) * CKV_D) : "memory");
  if (append && u_first < units) {
    const uint4 *src = reinterpret_cast<const uint4 *>((lane < 16 ? k_new : v_new) + (size_t)u_first * CKV_D);
#pragma unroll
    for (int k = 0; k < PP; ++k) piece[k] = __ldg(src + li + 16 * k);
  }
  auto eff_len = [&](int raw) { return max(min(raw + ((append && raw >= 0 && raw < cap) ? 1 : 0), cap), 0); };
  if (tid < batch) s_len[tid] = eff_len(len_mine);
  for (int i = tid + kThreads; i < batch && i < kMaxSeqs; i += kThreads) s_len[i] = eff_len(seq_lens[i]);
  __syncthreads();
  auto len_of = [&](int i) { return seq_len_of(P, s_len, seq_lens, i); };

  // The length before the append, from the staged (already incremented and clamped) one; the device array is only
  // asked where that is ambiguous (an empty or exactly full sequence).
  auto raw_len = [&](int sq_idx) {
    const int eff = len_of(sq_idx);
    return (eff > 0 && eff < cap && sq_idx < kMaxSeqs) ? eff - 1 : seq_lens[sq_idx];
  };
#pragma unroll 1
  for (int u = u_first; u < units; u += n_tail * 8) {
    const int s = ckv_div_hkv(P, u), h = u - s * P.Hkv;
    const int *pt_row = fresh.page_table + (size_t)s * P.max_pages_per_seq;
    const int raw = append ? raw_len(s) : -1;
    const bool room = raw >= 0 && raw < cap;
    int phys = -1;
    // the page of the new token is asked for first, and the unit's place among the scan partials (which depends on
    // the lengths only) is worked out while that entry is on its way
    if (append && room) phys = pt_row[raw / CKV_PAGE];
    int first = 0, count = 0;
    unit_scan_entries(P, len_of, units, u, nscan, lane, first, count);
    if (append) {
      if (!room) {
        if (lane == 0) atomicOr(P.status, CKV_DEV_SEQ_FULL);
      } else {
        const int slot = raw % CKV_PAGE;
        const int b = raw >> P.lg_bs, cnt = raw + 1 - b * P.bs;
        if (phys >= 0 && phys < P.num_pages) {
          if (u != u_first) {
            const uint4 *src = reinterpret_cast<const uint4 *>((lane < 16 ? k_new : v_new) + (size_t)u * CKV_D);
#pragma unroll
            for (int k = 0; k < PP; ++k) piece[k] = __ldg(src + li + 16 * k);
          }
          uint4 *dst = reinterpret_cast<uint4 *>((lane < 16 ? k_pool : v_pool) +
                                                 (((size_t)phys * P.Hkv + h) * CKV_PAGE + slot) * CKV_D);
#pragma unroll
          for (int k = 0; k < PP; ++k) dst[li + 16 * k] = piece[k];
        }
        __syncwarp();
        const size_t row = (size_t)u * P.max_blocks + b;
        // rows staged in this warp's slice of the (otherwise unused) ring memory when it is large enough
        constexpr int kStageBytes = 2 * CKV_PAGE * CKV_D * (int)sizeof(QT);
        if (smem_bytes >= 8 * CKV_D * 4 + 8 * kStageBytes)
          block_stats_warp_staged<QT>(P, k_pool, v_pool, pt_row, h, b, cnt,
                                      reinterpret_cast<unsigned char *>(smem_f + 8 * CKV_D) + (size_t)warp * kStageBytes, sq,
                                      P.kmean + row * P.row_elems, P.dbar + row * P.r, P.vmean + row * P.row_elems, lane);
        else
          block_stats_warp<QT, false>(P, k_pool, v_pool, pt_row, h, b, cnt, sq, P.kmean + row * P.row_elems,
                                      P.dbar + row * P.r, P.vmean + row * P.row_elems, lane);
      }
    }
    const int N = len_of(s);
    if (N == 0) continue;   // warp-uniform
    const int b = ((N + P.bs - 1) >> P.lg_bs) - 1, cnt = N - b * P.bs;
    const size_t row = (size_t)u * P.max_blocks + b;
    __syncwarp();
    float kx[8], vx[8], dx[8];   // this lane's 8 coordinates of kbar, vbar and of the variance of their group
    load_split8<false>(P.kmean + row * P.row_elems, li, b, kx, lo_half);
    load_split8<false>(P.vmean + row * P.row_elems, li, b, vx, lo_half && !P.vhi);   // as the scan CTAs read it
    if (P.r == CKV_D) {
      load_split8<false>(reinterpret_cast<const __nv_bfloat16 *>(P.dbar + row * CKV_D), li, b, dx);
    } else {
      // group of coordinate c: c / (128 / r), or ((c mod 64) / (64 / r)) in the half-split layout; r is a power of two
      const float *drow = P.dbar + row * P.r;
      const int sh = 31 - __clz(CKV_D / P.r);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = 8 * li + i;
        dx[i] = drow[P.glayout == 0 ? c >> sh : (c & (CKV_D / 2 - 1)) >> (sh - 1)];
      }
    }
    float *part = P.comp_part + (size_t)(first + count - 1) * G * CKV_PART_STRIDE;
    const float logc = logf((float)cnt);
#pragma unroll 1
    for (int g = 0; g < G; ++g) {
      float qx[8];   // this lane's 8 coordinates of query row u G + g
      load8<true>(q + ((size_t)u * G + g) * CKV_D + 8 * li, qx);
      float d = 0.f, sg = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        d = fmaf(qx[i], kx[i], d);
        const float qs = qx[i] * P.scale;
        sg = fmaf(qs * qs, dx[i], sg);   // Eq. 8: the squared logit scale is its 1/d
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) {
        d += __shfl_xor_sync(0xffffffffu, d, o);
        sg += __shfl_xor_sync(0xffffffffu, sg, o);
      }
      sg = fmaxf(sg, 0.f);
      const float zbar = d * P.scale;
      const float ell = logc + zbar + P.half_var * sg;
      const float zl2 = (zbar + logc) * kLog2e;
      float *pg = part + g * CKV_PART_STRIDE;
      if (lane == 0) {
        const size_t o = ((size_t)u * G + g) * P.max_blocks + b;
        P.lu[o] = fmaf(ell, kLog2e, by_mass ? 0.f : __log2f(sg));
        P.lz[o] = zl2;
        pg[0] = zl2; pg[1] = 1.f; pg[2] = fast_exp2(P.half_var * kLog2e * sg);   // maximum, weight 1, e^{l - m}
      }
      if (hw == 1) {   // weight 1 times the mean value
        *reinterpret_cast<float4 *>(pg + 4 + 8 * li) = make_float4(vx[0], vx[1], vx[2], vx[3]);
        *reinterpret_cast<float4 *>(pg + 8 + 8 * li) = make_float4(vx[4], vx[5], vx[6], vx[7]);
      }
    }
  }
}

template <typename QT> struct QSplit { static constexpr bool value = false; };
template <> struct QSplit<float> { static constexpr bool value = true; };

// RD: one variance group per coordinate (r = d).  The variance rows then have the mean rows' layout and
// sigma^2 = sum_i (scale q_i)^2 Dbar_i is a third tensor-core product, with the squared queries as the A operand.
// HS: the mean rows hold hi halves only (bf16 summaries, 256-byte rows); every product with a lo plane drops out.
// VH: full-precision rows in memory, but only the hi halves of the mean VALUES are brought in: one tensor copy per
// tile takes the first 256 bytes of each 512-byte row, and the value product is that of HS (Sec. 3.1: the
// compensation term is an average over many blocks; its rounding, at most half a bf16 step per block and of varying sign, is within that of the
// bf16 output).
template <int G, typename QT, bool RD, bool HS, bool VH>
__global__ void __launch_bounds__(kThreads, 1)
ckv_scan_kernel(CkvDev P, const QT *__restrict__ q, const int *seq_lens, int units, int stages, CkvNewToken fresh,
                int n_tail, const __grid_constant__ CUtensorMap tm_v) {
  constexpr bool QS = QSplit<QT>::value;   // fp32 queries are split into hi + lo like the summaries
  static_assert(!(VH && (HS || RD)), "VH is a variant of the full-precision layout with four variance groups");
  constexpr int kRowBytes = HS ? CKV_D * 2 : CKV_ROW_ELEMS * 2;   // bytes of one mean-key row in a stage
  constexpr int kRowBytesV = (HS || VH) ? CKV_D * 2 : CKV_ROW_ELEMS * 2;   // ... of one mean-value row
  constexpr int TB = ScanTile<HS || VH>::TB;
  extern __shared__ __align__(128) unsigned char stage_mem[];
  __shared__ __align__(8) uint64_t full_bar[2][kMaxStages], empty_bar[kMaxStages];
  __shared__ __align__(16) unsigned char s_zero_row[512];   // what mean-value rows past a unit's last block are read as
  __shared__ int s_u0, s_tl0, s_count, s_ulast, s_abort, s_issued;
  __shared__ int s_len[kMaxSeqs];
  // Query rows and variance weights of the first kStagedUnits units of this CTA's range (a CTA's range rarely
  // spans more than two), staged by the consumer warps while the first fills are on their way: a warp that moves
  // on to another unit then sets up from shared memory instead of paying a round trip to global memory.
  constexpr int kStagedUnits = 4;
  __shared__ __align__(16) __nv_bfloat16 s_q[kStagedUnits][G][CKV_D];
  __shared__ float s_w[kStagedUnits][G][4];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool r4 = P.r == 4;          // the default: the variance projection is four FMAs on one 16-byte read
  const bool dbar_bulk = P.r >= 4;   // smaller rows cannot keep the 16-byte alignment bulk copies need
  constexpr int kParts = TB / 16;    // 16-block parts of a tile, each worked on by one consumer warp
  const int stage_bytes = TB * (kRowBytes + kRowBytesV) + (dbar_bulk ? TB * P.r * 4 : 0);
  // per-warp w_{g,t} table for r != 4, behind the ring
  float *sw_all = reinterpret_cast<float *>(stage_mem + (size_t)stages * stage_bytes);

  // the sequence lengths are requested first; the ring is cleared while they are on their way
  const int batch = ckv_div_hkv(P, units);
  const bool append = fresh.k_new != nullptr;
  const int cap = P.max_blocks * P.bs;
  // length the step works on: one more than stored when a token is being appended (a full sequence keeps its length)
  auto eff_len = [&](int raw) { return max(min(raw + ((append && raw >= 0 && raw < cap) ? 1 : 0), cap), 0); };
  const int len_mine = tid < batch ? seq_lens[tid] : 0;
  if ((int)blockIdx.x < n_tail) {
    // ---------------- tail CTAs: the new token and the last block of every unit ----------------
    scan_tail<G, QT>(P, q, seq_lens, s_len, len_mine, units, (int)gridDim.x - n_tail, fresh, n_tail,
                     reinterpret_cast<float *>(stage_mem), stages * stage_bytes);
    if (append) lens_arrive(P.status + kLenCounter, seq_lens, fresh.seq_lens, batch, cap, (int)gridDim.x, /*whole_cta=*/true);
    return;
  }
  const int bid = (int)blockIdx.x - n_tail, nscan = (int)gridDim.x - n_tail;   // this CTA among the scan CTAs
  // rows of a stage past a unit's last block are never copied and the ring is never cleared: the products over
  // blocks read such mean-value rows from a row of zeros instead (a stale NaN pattern times a zero weight would
  // poison the accumulators); everywhere else a block is an output column, and those columns are discarded
  if (tid < 32) reinterpret_cast<uint4 *>(s_zero_row)[tid] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {   // also done while the lengths are on their way: the barriers of the ring
    for (int st = 0; st < stages; ++st) { mbar_init(&full_bar[0][st], 1); mbar_init(&full_bar[1][st], 1); mbar_init(&empty_bar[st], kParts); }
    fence_barrier_init();
  }
  if (tid < batch) s_len[tid] = eff_len(len_mine);
  for (int i = tid + kThreads; i < batch && i < kMaxSeqs; i += kThreads) s_len[i] = eff_len(seq_lens[i]);
  __syncthreads();
  if (tid == 0) {
    // this CTA's range of the tiles (a step has fewer than 2^24 tiles, checked at creation: ckv_udiv24)
    unsigned T = 0;
    for (int i = 0; i < batch; ++i) T += (unsigned)seq_tiles(s_len, seq_lens, P, i) * (unsigned)P.Hkv;
    const unsigned tpc = ckv_udiv24(T + (unsigned)nscan - 1u, (unsigned)nscan);
    const unsigned first = (unsigned)bid * tpc;
    const unsigned cnt = first >= T ? 0u : min(T - first, tpc);
    int u0 = 0, tl0 = 0, ulast = 0;
    if (cnt > 0) {
      unsigned accum = 0;
      bool have_first = false;
      for (int i = 0; i < batch; ++i) {
        const unsigned t = (unsigned)seq_tiles(s_len, seq_lens, P, i);
        if (t > 0) {
          if (!have_first && first < accum + t * (unsigned)P.Hkv) {
            const unsigned off = first - accum;
            const unsigned oq = ckv_udiv24(off, t);
            u0 = i * P.Hkv + (int)oq; tl0 = (int)(off - oq * t);
            have_first = true;
          }
          if (first + cnt - 1u < accum + t * (unsigned)P.Hkv) {
            ulast = i * P.Hkv + (int)ckv_udiv24(first + cnt - 1u - accum, t);
            break;
          }
        }
        accum += t * (unsigned)P.Hkv;
      }
    }
    s_u0 = u0; s_tl0 = tl0; s_ulast = ulast; s_count = (int)cnt; s_abort = 0; s_issued = 0;
  }
  __syncthreads();
  const int count = s_count;
  // Every length this CTA needs is in shared memory now: one thread says so (the last CTA of the grid to say it
  // stores the new lengths).  It is a spare lane of the producer warp, in the same if/else as the producer, so
  // that nobody waits for its round trip.
  if (count == 0) {   // uniform: this CTA has no tiles
    if (append && tid == kThreads - 1) lens_arrive(P.status + kLenCounter, seq_lens, fresh.seq_lens, batch, cap, (int)gridDim.x, false);
    return;
  }

  if (warp == kConsumerWarps) {
    // ---------------- producer: one thread streams the CTA's tiles into the ring ----------------
    if (lane == 0) {
      int u = s_u0, tl = s_tl0, st = 0;
      uint32_t phase = 0;            // parity of the empty-barrier phase the next refill of stage `st` waits for
      uint32_t round = 0;            // times the ring has wrapped: fill `it` uses the full barrier [round & 1][st]
      UnitInfo ui = unit_info(P, s_len, seq_lens, u);
      for (int it = 0; it < count; ++it) {
        if (it >= stages && !mbar_wait(&empty_bar[st], phase, P.spin_limit)) {
          atomicOr(P.status, CKV_DEV_TIMEOUT);
          *(volatile int *)&s_abort = 1;
        }
        if (*(volatile int *)&s_abort) break;
        const int b0 = tl * TB;
        const int nb = min(TB, ui.X - b0);
        const size_t row = (size_t)u * P.max_blocks + b0;
        unsigned char *sk = stage_mem + (size_t)st * stage_bytes;
        unsigned char *sv = sk + TB * kRowBytes;
        const uint32_t kbytes = (uint32_t)nb * kRowBytes;
        const uint32_t dbytes = dbar_bulk ? (uint32_t)nb * P.r * 4 : 0;
        uint64_t *fb = &full_bar[round & 1][st];
        const uint32_t vbytes = VH ? (uint32_t)TB * kRowBytesV : kbytes;   // a tensor copy always delivers its whole box
        mbar_arrive_expect_tx(fb, kbytes + vbytes + dbytes);
        const uint32_t lo = smem_u32(stage_mem), hi = lo + (uint32_t)stages * stage_bytes;
        bool ok = nb >= 1 && u < units && row + nb <= (size_t)units * P.max_blocks;
        // test hook (ckv_debug_set): one fill is announced but never issued, so that the waits on it run out
        const bool skip = (P.debug & CKV_DEBUG_SKIP_FILL) != 0 && it == 0 && bid == 0;
        if (!skip) {
          ok = ok && bulk_g2s_checked(sk, P.kmean + row * P.row_elems, kbytes, fb, lo, hi);
          if constexpr (VH) {
            // rows [row, row + TB) of the mean-values region, first 256 bytes of each (rows past the unit's blocks are
            // never read; rows past the region's end arrive as zeros)
            const uint32_t dv = smem_u32(sv);
            const bool fits = (dv & 127u) == 0 && dv >= lo && dv + vbytes <= hi;
            if (ok && fits) tensor_g2s(dv, &tm_v, 0, (int)row, fb);
            ok = ok && fits;
          } else {
            ok = ok && bulk_g2s_checked(sv, P.vmean + row * P.row_elems, kbytes, fb, lo, hi);
          }
          if (dbar_bulk) ok = ok && bulk_g2s_checked(sv + TB * kRowBytesV, P.dbar + row * P.r, dbytes, fb, lo, hi);
          *(volatile int *)&s_issued = it + 1;
        }
        if (!ok) atomicOr(P.status, CKV_DEV_BAD_COPY);
        if (++st == stages) { st = 0; ++round; if (it >= stages) phase ^= 1; }
        if (++tl == ui.tiles) {
          tl = 0;
          do { ++u; } while (u < units && (ui = unit_info(P, s_len, seq_lens, u)).tiles == 0);
        }
      }
    } else if (append && lane == 31) {
      lens_arrive(P.status + kLenCounter, seq_lens, fresh.seq_lens, batch, cap, (int)gridDim.x, false);
    }
  } else {
    // ---------------- consumer warps: half tile j = warp, warp + 8, ... of the CTA's range ----------------
    const int head = lane >> 2, qd = lane & 3;   // this thread's accumulator row (head) and column pair
    const bool hv = head < G;
    constexpr bool SP = (G <= 4) && !RD;   // the per-(head, block) arithmetic is shared between the half warps
    constexpr int NE = SP ? 1 : 2;          // n-tiles a lane works on there
    const int hsel = lane >> 4;             // ... and which one: the lower half warp the first, the upper the second
    const int ehead = SP ? (head & 3) : head;
    const bool ehv = ehead < G;
    const bool staged = !QS && !RD && P.r == 4;   // bf16 queries, four variance groups: the staged setup below
    if (staged) {
      constexpr int kPieces = G * CKV_D * 2 / 16;   // 16-byte pieces of a unit's G query rows
      for (int idx = tid; idx < kStagedUnits * kPieces; idx += kConsumerWarps * 32) {
        const int k = idx / kPieces, pc = idx % kPieces, uu = s_u0 + k;
        if (uu <= s_ulast && uu < units) {
          const int s2 = ckv_div_hkv(P, uu), h2 = uu - s2 * P.Hkv;
          const uint4 *src = reinterpret_cast<const uint4 *>(q + ((size_t)s2 * P.Hq + h2 * G) * CKV_D);
          reinterpret_cast<uint4 *>(&s_q[k][0][0])[pc] = __ldg(src + pc);
        }
      }
      named_barrier(1, kConsumerWarps * 32);
      // w_{g,t} of Eq. 8: sums of squared query coordinates per variance group, times the squared logit scale
      for (int idx = tid; idx < kStagedUnits * G * 4; idx += kConsumerWarps * 32) {
        const int k = idx / (G * 4), g = (idx / 4) % G, t = idx % 4;
        if (s_u0 + k <= s_ulast) {
          float w = 0.f;
          for (int i = 0; i < CKV_D / 4; ++i) {   // the group's 32 coordinates: one run, or two runs of 16
            const int c = P.glayout == 0 ? 32 * t + i : (i < 16 ? 16 * t + i : CKV_D / 2 + 16 * t + (i - 16));
            const float x = __bfloat162float(s_q[k][g][c]);
            w = fmaf(x, x, w);
          }
          s_w[k][g][t] = w * (P.scale * P.scale);
        }
      }
      named_barrier(1, kConsumerWarps * 32);
    }
    uint32_t qa[8][2], qb[QS ? 8 : 1][2];        // A fragments of the unit's queries (rows 0..7), per 16-coordinate step
    uint32_t qsh[RD ? 8 : 1][2], qsl[RD ? 8 : 1][2];   // (scale q)^2 as hi and lo halves, same fragment positions
    float acc[16][2];                            // W Vbar accumulator: head `head`, coordinates 8 t + 2 qd + {0, 1}
    float m_ref = -CUDART_INF_F, l_acc = 0.f, lp_acc = 0.f;
    float wown[4] = {0.f, 0.f, 0.f, 0.f};
    float *sw = sw_all + (size_t)warp * P.r * G;   // [t][g], r != 4 only
    const float log_bs = logf((float)P.bs);
    const bool by_mass = (P.variant & CKV_VARIANT_RANK_BY_MASS) != 0;
    float log_last = 0.f;   // log of the token count of the unit's last block, when the scan CTAs cover it
    const bool pair_ok = (P.max_blocks & 1) == 0;   // rows of the per-block outputs start on 8-byte boundaries
    const int ulast = s_ulast;
    int u = s_u0, tl = s_tl0, cur = -1, next_empty = s_u0;
    UnitInfo ui = unit_info(P, s_len, seq_lens, u);
    float *lu = nullptr, *lz = nullptr;
    const float *db = nullptr;
    bool aborted = false;

    auto write_partial = [&](int unit_id, bool real) {
      float *part = P.comp_part + ((size_t)(bid + 2 * unit_id) * kConsumerWarps + warp) * G * CKV_PART_STRIDE;
      if (!real) {
        if (lane < G) {
          part[lane * CKV_PART_STRIDE] = -CUDART_INF_F;
          part[lane * CKV_PART_STRIDE + 1] = 0.f;
          part[lane * CKV_PART_STRIDE + 2] = 0.f;
        }
        return;
      }
      // l and lp: sum over the four lanes that share the head
      float l = l_acc, lp = lp_acc;
      l += __shfl_xor_sync(0xffffffffu, l, 1); l += __shfl_xor_sync(0xffffffffu, l, 2);
      lp += __shfl_xor_sync(0xffffffffu, lp, 1); lp += __shfl_xor_sync(0xffffffffu, lp, 2);
      if (SP) { l += __shfl_xor_sync(0xffffffffu, l, 16); lp += __shfl_xor_sync(0xffffffffu, lp, 16); }
      if (hv) {
        float *pg = part + head * CKV_PART_STRIDE;
#pragma unroll
        for (int t = 0; t < 16; ++t)
          *reinterpret_cast<float2 *>(pg + 4 + 8 * t + 2 * qd) = make_float2(acc[t][0], acc[t][1]);
        if (qd == 0) { pg[0] = m_ref; pg[1] = l; pg[2] = lp; }
      }
    };
    // units of this CTA's range that this warp never worked on still need an (empty) partial
    auto fill_empty_upto = [&](int upto) {
      for (; next_empty < upto; ++next_empty)
        if (unit_info(P, s_len, seq_lens, next_empty).tiles > 0) write_partial(next_empty, false);
    };

    // Part j = kParts * tile + part-of-tile belongs to warp j % W, and a warp visits only the tiles that hold one
    // of its parts: it waits for the tile's fill, works on its part and releases the stage; a stage is refilled
    // once the kParts owners of its parts have released it.  A warp's next part is at most W parts (four tiles)
    // ahead, and fill f is only issued after fill f - stages has landed and been released, so the stage a warp
    // waits on is at most two fills behind the one it wants.  A parity wait can only tell a fill from the one
    // before it, hence the two sets of full barriers used by alternate rounds of the ring: together they tell four
    // consecutive fills of a stage apart.
    int it_at = 0;   // tile the (u, tl) walk stands at
    uint32_t round = 0;   // the tile's place in the ring, kept by stepping (a division per visit would be two dozen instructions)
    int st = 0;
    for (int pidx = warp; pidx < kParts * count; pidx += kConsumerWarps) {
      const int it = pidx / kParts;
      int half = pidx - it * kParts;
      st += it - it_at;
      while (st >= stages) { st -= stages; ++round; }
      for (; it_at < it; ++it_at) {
        if (++tl == ui.tiles) {
          tl = 0;
          do { ++u; } while (u < units && (ui = unit_info(P, s_len, seq_lens, u)).tiles == 0);
        }
      }
      // a wait that runs out marks the step invalid (`aborted`); the walk still runs to the end
      if (!aborted) {
        bool fail = *(volatile int *)&s_abort != 0;
        if (!fail && !mbar_wait(&full_bar[round & 1][st], (round >> 1) & 1, P.spin_limit)) {
          atomicOr(P.status, CKV_DEV_TIMEOUT);
          *(volatile int *)&s_abort = 1;
          fail = true;
        }
        aborted = __any_sync(0xffffffffu, fail);
      }
      if (half >= 0) {
      if (u != cur) {
        if (cur >= 0) { write_partial(cur, true); next_empty = cur + 1; }
        fill_empty_upto(u);
        // per-unit setup: query fragments, variance weights, fresh accumulators
        const int s = ckv_div_hkv(P, u), h = u - s * P.Hkv;
        const QT *qrow = q + ((size_t)s * P.Hq + h * G + (hv ? head : 0)) * CKV_D;
        const int uk = u - s_u0;
        const bool from_smem = staged && uk < kStagedUnits;
        if (from_smem) {
          const uint32_t *srow = reinterpret_cast<const uint32_t *>(&s_q[uk][hv ? head : 0][0]);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) qa[ks][hh] = hv ? srow[(16 * ks + 8 * hh + 2 * qd) / 2] : 0u;
#pragma unroll
          for (int t = 0; t < 4; ++t) wown[t] = ehv ? s_w[uk][ehead][t] : 0.f;
        } else {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int c0 = 16 * ks + 8 * hh + 2 * qd;
            const float x0 = hv ? to_float(qrow[c0]) : 0.f, x1 = hv ? to_float(qrow[c0 + 1]) : 0.f;
            qa[ks][hh] = pack_bf16(x0, x1);
            if (QS) qb[QS ? ks : 0][hh] = pack_bf16(x0 - bf16_round(x0), x1 - bf16_round(x1));
            if (RD) {
              const float s0 = (x0 * P.scale) * (x0 * P.scale), s1 = (x1 * P.scale) * (x1 * P.scale);
              qsh[RD ? ks : 0][hh] = pack_bf16(s0, s1);
              qsl[RD ? ks : 0][hh] = pack_bf16(s0 - bf16_round(s0), s1 - bf16_round(s1));
            }
          }
        }
        }
        if (from_smem) {
          // set up above
        } else if (RD) {
          // nothing to tabulate: the weights are the squared queries held above
        } else if (r4) {
          // w_{g,t} for this thread's head: every lane of the quad sums all 128 coordinates (once per unit)
          float wsum[4] = {0.f, 0.f, 0.f, 0.f};
          const QT *qrow_e = q + ((size_t)s * P.Hq + h * G + (ehv ? ehead : 0)) * CKV_D;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float x[8];
            load8<true>(qrow_e + 8 * c, x);
            float s8 = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) s8 = fmaf(x[i], x[i], s8);
            // an aligned run of 8 coordinates lies in one group for r = 4 (groups are runs of 32 or 16)
            const int t = P.glayout == 0 ? (8 * c) / 32 : ((8 * c) % 64) / 16;
            wsum[0] += t == 0 ? s8 : 0.f; wsum[1] += t == 1 ? s8 : 0.f;
            wsum[2] += t == 2 ? s8 : 0.f; wsum[3] += t == 3 ? s8 : 0.f;
          }
          if (!ehv) { wsum[0] = wsum[1] = wsum[2] = wsum[3] = 0.f; }
#pragma unroll
          for (int t = 0; t < 4; ++t) wown[t] = wsum[t] * (P.scale * P.scale);   // Eq. 8's 1/d is the squared logit scale
        } else {
          __syncwarp();
          for (int idx = lane; idx < P.r * G; idx += 32) {
            const int t = idx / G, g = idx % G;
            const QT *qg = q + ((size_t)s * P.Hq + h * G + g) * CKV_D;
            float w = 0.f;
            for (int i = 0; i < CKV_D; ++i)
              if (group_of(i, P.r, P.glayout) == t) { const float x = to_float(qg[i]); w = fmaf(x, x, w); }
            sw[idx] = w * (P.scale * P.scale);
          }
          __syncwarp();
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) { acc[t][0] = 0.f; acc[t][1] = 0.f; }
        m_ref = -CUDART_INF_F; l_acc = 0.f; lp_acc = 0.f;
        log_last = logf((float)(ui.N - (ui.X - 1) * P.bs));
        const size_t row0 = (size_t)u * P.max_blocks;
        lu = P.lu + row0 * G;   // [head][block] within the unit
        lz = P.lz + row0 * G;
        db = P.dbar + row0 * P.r;
        cur = u;
      }
      const int b0 = tl * TB;
      const int nb = min(TB, ui.X - b0);
      const int rb = half * 16;          // first row of this warp's half tile
      if (!aborted && rb < nb) {
        const uint32_t sk = smem_u32(stage_mem + (size_t)st * stage_bytes);
        const uint32_t sv = sk + TB * kRowBytes;
        const float *sd = reinterpret_cast<const float *>(stage_mem + (size_t)st * stage_bytes + TB * (kRowBytes + kRowBytesV));

        // ---- Z^T = Q Kbar^T: heads x 16 blocks (two n-tiles of 8 blocks), hi and lo planes into one accumulator ----
        // four accumulation chains per n-tile (hi / lo plane x even / odd 16-coordinate step): the products of a chain
        // depend on one another, and a warp has little else to issue while it waits for them
        float z[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, zlo[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        float z2[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, zlo2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        {
          // ldmatrix lane roles: matrix lane / 8 -> 8-coordinate chunk, row lane % 8
          const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const int r = rb + nt * 8 + lrow;
            const uint32_t rowaddr = sk + r * kRowBytes;
#pragma unroll
            for (int j = 0; j < 4; ++j) {   // two 16-coordinate steps per ldmatrix.x4
              const uint32_t coff = (uint32_t)swz_chunk(4 * j + lmat, r) * 16;
              uint32_t bh[4], bl[4];
              ldmatrix_x4(bh, rowaddr + coff);
              mma_rows8(z[nt][0], z[nt][1], qa[2 * j][0], qa[2 * j][1], bh[0], bh[1]);
              mma_rows8(z2[nt][0], z2[nt][1], qa[2 * j + 1][0], qa[2 * j + 1][1], bh[2], bh[3]);
              if (!HS) {
                ldmatrix_x4(bl, rowaddr + 256 + coff);
                mma_rows8(zlo[nt][0], zlo[nt][1], qa[2 * j][0], qa[2 * j][1], bl[0], bl[1]);
                mma_rows8(zlo2[nt][0], zlo2[nt][1], qa[2 * j + 1][0], qa[2 * j + 1][1], bl[2], bl[3]);
              }
              if (QS) {
                mma_rows8(zlo[nt][0], zlo[nt][1], qb[QS ? 2 * j : 0][0], qb[QS ? 2 * j : 0][1], bh[0], bh[1]);
                mma_rows8(zlo[nt][0], zlo[nt][1], qb[QS ? 2 * j + 1 : 0][0], qb[QS ? 2 * j + 1 : 0][1], bh[2], bh[3]);
              }
            }
            z[nt][0] = (z[nt][0] + z2[nt][0]) + (zlo[nt][0] + zlo2[nt][0]);
            z[nt][1] = (z[nt][1] + z2[nt][1]) + (zlo[nt][1] + zlo2[nt][1]);
          }
        }
        float sgm[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        if (RD) {   // sigma^2 for the same heads x blocks tile: (qs_hi + qs_lo) (D_hi + D_lo) without the lo lo term
          float sg2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
          const uint32_t sdr = sv + TB * kRowBytes;
          const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const int r = rb + nt * 8 + lrow;
            const uint32_t rowaddr = sdr + r * kRowBytes;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t coff = (uint32_t)swz_chunk(4 * j + lmat, r) * 16;
              uint32_t dh[4], dl[4];
              ldmatrix_x4(dh, rowaddr + coff);
              ldmatrix_x4(dl, rowaddr + 256 + coff);
              mma_rows8(sgm[nt][0], sgm[nt][1], qsh[RD ? 2 * j : 0][0], qsh[RD ? 2 * j : 0][1], dh[0], dh[1]);
              mma_rows8(sgm[nt][0], sgm[nt][1], qsh[RD ? 2 * j + 1 : 0][0], qsh[RD ? 2 * j + 1 : 0][1], dh[2], dh[3]);
              mma_rows8(sg2[nt][0], sg2[nt][1], qsl[RD ? 2 * j : 0][0], qsl[RD ? 2 * j : 0][1], dh[0], dh[1]);
              mma_rows8(sg2[nt][0], sg2[nt][1], qsl[RD ? 2 * j + 1 : 0][0], qsl[RD ? 2 * j + 1 : 0][1], dh[2], dh[3]);
              mma_rows8(sg2[nt][0], sg2[nt][1], qsh[RD ? 2 * j : 0][0], qsh[RD ? 2 * j : 0][1], dl[0], dl[1]);
              mma_rows8(sg2[nt][0], sg2[nt][1], qsh[RD ? 2 * j + 1 : 0][0], qsh[RD ? 2 * j + 1 : 0][1], dl[2], dl[3]);
            }
            sgm[nt][0] += sg2[nt][0]; sgm[nt][1] += sg2[nt][1];
          }
        }

        // ---- per (head, block): variance projection, l, running maximum, compensation weight ----
        // The products leave this part's 16 blocks x G heads in the lanes of rows 0..G-1 (four values per lane).
        // With G <= 4 those are lanes 0-15 only, so the upper half warp takes over the second n-tile: every lane
        // then works on one n-tile's pair of blocks (half the dependent chain), and the weights travel back to
        // the lower lanes, which hold the A operand of the next product.
        float zin[NE][2];
        if constexpr (SP) {
          const float t0 = __shfl_sync(0xffffffffu, z[1][0], lane & 15), t1 = __shfl_sync(0xffffffffu, z[1][1], lane & 15);
          zin[0][0] = hsel ? t0 : z[0][0];
          zin[0][1] = hsel ? t1 : z[0][1];
        } else {
#pragma unroll
          for (int k = 0; k < NE; ++k) { zin[k][0] = z[k][0]; zin[k][1] = z[k][1]; }
        }
        float zl2[NE][2], sig[NE][2], wt[NE][2];
        bool val[NE][2];
        float tmax = -CUDART_INF_F;
#pragma unroll
        for (int k = 0; k < NE; ++k) {
          const int nt = SP ? hsel : k;
          const int r0 = rb + nt * 8 + 2 * qd;     // this thread's two blocks of the n-tile: rows r0, r0 + 1
          float ell[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int r = r0 + e, b = b0 + r;
            val[k][e] = ehv && r < nb;
            float sg = 0.f;
            if (val[k][e]) {
              if (RD) {
                sg = fmaxf(sgm[RD ? k : 0][e], 0.f);
              } else if (r4) {
                const float4 dv = *reinterpret_cast<const float4 *>(sd + r * 4);
                sg = fmaf(wown[0], dv.x, fmaf(wown[1], dv.y, fmaf(wown[2], dv.z, wown[3] * dv.w)));
              } else {
                for (int t = 0; t < P.r; ++t) {
                  const float dv = dbar_bulk ? sd[r * P.r + t] : __ldg(db + (size_t)b * P.r + t);
                  sg = fmaf(sw[t * G + ehead], dv, sg);
                }
              }
            }
            sig[k][e] = sg;
            const float zbar = zin[k][e] * P.scale;
            const float logc = (!P.tail && b == ui.X - 1) ? log_last : log_bs;   // in tail mode every block here is full
            ell[e] = logc + zbar + P.half_var * sg;
            zl2[k][e] = val[k][e] ? (zbar + logc) * kLog2e : -CUDART_INF_F;   // log2 of |b| e^{zbar}
            tmax = fmaxf(tmax, zl2[k][e]);
          }
          // what the later kernels read, both in log2 units: the head's term of the block score, e^l sigma^2 (e^l
          // alone when blocks are ranked by mass), and the block's mean-compensation weight |b| e^{zbar}.  The
          // thread's two blocks are neighbours: one 8-byte store each when the rows are 8-byte aligned.
          const size_t o = (size_t)ehead * P.max_blocks + b0 + r0;
          const float u0 = fmaf(ell[0], kLog2e, by_mass ? 0.f : __log2f(sig[k][0]));
          const float u1 = fmaf(ell[1], kLog2e, by_mass ? 0.f : __log2f(sig[k][1]));
          if (pair_ok && val[k][1]) {
            *reinterpret_cast<float2 *>(lu + o) = make_float2(u0, u1);
            *reinterpret_cast<float2 *>(lz + o) = make_float2(zl2[k][0], zl2[k][1]);
          } else {
            if (val[k][0]) { lu[o] = u0; lz[o] = zl2[k][0]; }
            if (val[k][1]) { lu[o + 1] = u1; lz[o + 1] = zl2[k][1]; }
          }
        }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        if (SP) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
        if (tmax > m_ref + CKV_RESCALE_SLACK) {   // the running maximum is only raised when exceeded by a slack
          const float sc = exp2_diff(m_ref, tmax);
          m_ref = tmax;
          l_acc *= sc; lp_acc *= sc;
#pragma unroll
          for (int t = 0; t < 16; ++t) { acc[t][0] *= sc; acc[t][1] *= sc; }
        }
        uint32_t whm[NE], wlm[NE];
#pragma unroll
        for (int k = 0; k < NE; ++k) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            wt[k][e] = val[k][e] ? fast_exp2(zl2[k][e] - m_ref) : 0.f;
            l_acc += wt[k][e];
            lp_acc = fmaf(wt[k][e], fast_exp2(P.half_var * kLog2e * sig[k][e]), lp_acc);   // e^{l - m} = e^{zbar + log|b| - m} e^{sigma^2/2}
          }
          whm[k] = pack_bf16(wt[k][0], wt[k][1]);
          wlm[k] = pack_bf16(wt[k][0] - bf16_round(wt[k][0]), wt[k][1] - bf16_round(wt[k][1]));
        }
        uint32_t wh[2], wl[2];   // A fragments of the weights: k = blocks 2 qd + {0, 1} (+ 8), hi and lo halves
        if constexpr (SP) {
          // rows 0..3 (lanes 0-15) get their second n-tile from the lane 16 above; rows 4..7 carry zero weights
          const uint32_t oh = __shfl_sync(0xffffffffu, whm[0], (lane & 15) + 16);
          const uint32_t ol = __shfl_sync(0xffffffffu, wlm[0], (lane & 15) + 16);
          wh[0] = hsel ? 0u : whm[0]; wl[0] = hsel ? 0u : wlm[0];
          wh[1] = hsel ? 0u : oh;     wl[1] = hsel ? 0u : ol;
        } else {
#pragma unroll
          for (int k = 0; k < NE; ++k) { wh[k] = whm[k]; wl[k] = wlm[k]; }
        }

        // ---- acc += W Vbar: heads x 128 coordinates, k = this half tile's 16 blocks ----
        {
          // ldmatrix.trans lane roles: matrix lane / 8 -> (block half, coordinate chunk parity), row lane % 8
          const int r = rb + ((lane >> 3) & 1) * 8 + (lane & 7);
          const bool real = r < nb;   // rows past the unit's last block: zeros
          const uint32_t rowaddr = real ? sv + r * kRowBytesV : smem_u32(s_zero_row);
          const int cpar = lane >> 4;
#pragma unroll
          for (int t2 = 0; t2 < 8; ++t2) {   // two 8-coordinate n-tiles per ldmatrix.x4
            const uint32_t coff = real ? (uint32_t)swz_chunk(2 * t2 + cpar, r) * 16 : 0u;
            uint32_t vh[4], vl[4];
            ldmatrix_x4_trans(vh, rowaddr + coff);
            mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh[0], wh[1], vh[0], vh[1]);
            mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wl[0], wl[1], vh[0], vh[1]);
            mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh[0], wh[1], vh[2], vh[3]);
            mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wl[0], wl[1], vh[2], vh[3]);
            if (!HS && !VH) {
              ldmatrix_x4_trans(vl, rowaddr + (real ? 256u : 0u) + coff);
              mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh[0], wh[1], vl[0], vl[1]);
              mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh[0], wh[1], vl[2], vl[3]);
            }
          }
        }
      }
      }   // own part
      __syncwarp();
      if (lane == 0 && !aborted) mbar_arrive(&empty_bar[st]);
    }
    if (cur >= 0) { write_partial(cur, true); next_empty = cur + 1; }
    fill_empty_upto(ulast + 1);
  }
  __syncthreads();
  if (s_abort && tid == 0) {
    // leave no bulk copy in flight into this CTA's shared memory: wait (bounded) for every issued fill
    // (a completed phase is seen as complete again, so waiting on consumed stages returns at once)
    const int issued = s_issued;
    for (int it = max(issued - stages, 0); it < issued; ++it)
      mbar_wait(&full_bar[(it / stages) & 1][it % stages], ((it / stages) >> 1) & 1, P.spin_limit);
  }
}

struct ScanCfg { int stages; size_t smem; };

ScanCfg scan_cfg(const CkvDev &P, int G) {
  const size_t TB = (size_t)P.scan_tile;
  const size_t krow = (size_t)P.row_elems * 2, vrow = P.vhi ? (size_t)CKV_D * 2 : krow;
  const size_t stage_bytes = TB * (krow + vrow) + (P.r >= 4 ? TB * P.r * 4 : 0);
  const size_t sw_bytes = (P.r == 4 || P.r == CKV_D) ? 0 : (size_t)kConsumerWarps * P.r * G * 4;   // weight table of the generic path
  // 227 KB per CTA, less the kernel's static shared memory (lengths, barriers, the row of zeros: under 6 KB; staged
  // query rows and variance weights: 4 units x G x 272 bytes) and a reserve
  const size_t stat = 6 * 1024 + (size_t)4 * G * (CKV_D * 2 + 16);
  const size_t budget = 227 * 1024 - stat - 1024 - sw_bytes;
  int stages = (int)(budget / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  // A consumer warp's next part is at most kConsumerWarps parts ahead of its last one; the ring protocol needs
  // that distance, in tiles, to be no more than the number of stages (see the consumer loop).
  const int parts = (int)TB / 16;
  const int need = (kConsumerWarps + parts - 1) / parts;
  if (stages < need) stages = 0;   // refused by the launcher (no layout reaches this on a 227 KB part)
  return ScanCfg{stages, stages * stage_bytes + sw_bytes};
}

template <int G, typename QT>
cudaError_t launch_gt(ckv_ctx *c, const void *q, const int *seq_lens, int units, int grid, const CkvNewToken &fresh,
                      int n_tail, cudaStream_t st) {
  const ScanCfg cfg = scan_cfg(c->dev, G);
  if (cfg.stages == 0) return cudaErrorInvalidConfiguration;
  if (c->dev.r == CKV_D)
    ckv_scan_kernel<G, QT, true, false, false><<<grid, kThreads, cfg.smem, st>>>(c->dev, (const QT *)q, seq_lens, units, cfg.stages, fresh, n_tail, c->tm_vhi);
  else if (c->dev.row_elems == CKV_D) {
    if constexpr (!QSplit<QT>::value)   // bf16 summaries come with bf16 pages and queries only
      ckv_scan_kernel<G, QT, false, true, false><<<grid, kThreads, cfg.smem, st>>>(c->dev, (const QT *)q, seq_lens, units, cfg.stages, fresh, n_tail, c->tm_vhi);
    else
      return cudaErrorInvalidValue;
  } else if (c->dev.vhi) {
    if constexpr (!QSplit<QT>::value)
      ckv_scan_kernel<G, QT, false, false, true><<<grid, kThreads, cfg.smem, st>>>(c->dev, (const QT *)q, seq_lens, units, cfg.stages, fresh, n_tail, c->tm_vhi);
    else
      return cudaErrorInvalidValue;
  } else
    ckv_scan_kernel<G, QT, false, false, false><<<grid, kThreads, cfg.smem, st>>>(c->dev, (const QT *)q, seq_lens, units, cfg.stages, fresh, n_tail, c->tm_vhi);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, const void *q, const int *seq_lens, int units, int grid, const CkvNewToken &fresh,
                     int n_tail, cudaStream_t st) {
  if (c->layout.kv_dtype == CKV_BF16) return launch_gt<G, __nv_bfloat16>(c, q, seq_lens, units, grid, fresh, n_tail, st);
  return launch_gt<G, float>(c, q, seq_lens, units, grid, fresh, n_tail, st);
}

template <int G, typename QT>
cudaError_t configure_gt(const ckv_ctx *c) {
  const int smem = (int)scan_cfg(c->dev, G).smem;
  if (c->dev.r == CKV_D)
    return cudaFuncSetAttribute(ckv_scan_kernel<G, QT, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (c->dev.row_elems == CKV_D) {
    if constexpr (!QSplit<QT>::value)
      return cudaFuncSetAttribute(ckv_scan_kernel<G, QT, false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return cudaErrorInvalidValue;
  }
  if (c->dev.vhi) {
    if constexpr (!QSplit<QT>::value)
      return cudaFuncSetAttribute(ckv_scan_kernel<G, QT, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return cudaErrorInvalidValue;
  }
  return cudaFuncSetAttribute(ckv_scan_kernel<G, QT, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

// The mean-values region as the copy engine sees it with vhi: a matrix of bf16 rows, [units * max_blocks][128] at a pitch
// of 512 bytes (the hi halves of the stored rows), copied in boxes of CKV_SCAN_TILE_HS rows.  Host-side arithmetic only;
// the encoder is the driver's, looked up once through the runtime.
cudaError_t make_vhi_map(ckv_ctx *c) {
  using encode_fn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static std::mutex mtx;
  static encode_fn encode = nullptr;
  {
    std::lock_guard<std::mutex> lock(mtx);
    if (encode == nullptr) {
      void *fn = nullptr;
      cudaDriverEntryPointQueryResult qres = cudaDriverEntryPointSymbolNotFound;
      const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
      if (e != cudaSuccess) return e;
      if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorSymbolNotFound;
      encode = reinterpret_cast<encode_fn>(fn);
    }
  }
  const CkvDev &P = c->dev;
  if (((uintptr_t)P.vmean & 15u) != 0) return cudaErrorMisalignedAddress;
  const cuuint64_t dims[2] = {(cuuint64_t)CKV_D, (cuuint64_t)c->layout.max_batch * P.Hkv * P.max_blocks};
  const cuuint64_t strides[1] = {(cuuint64_t)CKV_ROW_ELEMS * 2};   // bytes between rows
  const cuuint32_t box[2] = {CKV_D, CKV_SCAN_TILE_HS};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = encode(&c->tm_vhi, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)P.vmean, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int G>
cudaError_t configure_g(ckv_ctx *c) {
  if (c->dev.vhi) {
    const cudaError_t e = make_vhi_map(c);
    if (e != cudaSuccess) return e;
  }
  if (c->layout.kv_dtype == CKV_BF16) return configure_gt<G, __nv_bfloat16>(c);
  return configure_gt<G, float>(c);
}

}  // namespace

// Opt in to the dynamic shared memory this context's scan instantiation needs, on the current device.
cudaError_t ckv_configure_scan(ckv_ctx *c) {
  switch (c->dev.G) {
    case 1: return configure_g<1>(c);
    case 2: return configure_g<2>(c);
    case 4: return configure_g<4>(c);
    case 8: return configure_g<8>(c);
  }
  return cudaErrorInvalidValue;
}

namespace {
// Tail CTAs of a launch: 8 warps each, one unit per warp and round.  One round is the goal: a warp's work is a chain
// of three or four dependent cache misses, each of which costs several microseconds once the scan CTAs have
// saturated DRAM (two rounds for 32 units made the whole step 7 us slower than one).
int tail_ctas(const ckv_ctx *c, int batch) {
  if (!c->dev.tail) return 0;
  const int units = batch * c->dev.Hkv;
  const int one_round = (units + 7) / 8;
  if (one_round <= 16) return std::max(1, one_round);
  return std::min((units + 15) / 16, std::max(16, c->sm_count / 4));   // many units: two rounds, at most a quarter of the SMs
}
}  // namespace

// Scan CTAs of a step: one persistent CTA per SM the tail CTAs leave free, never more CTAs than tiles.
int ckv_scan_grid(const ckv_ctx *c, int batch, int max_len) {
  const CkvDev &P = c->dev;
  const int xmax = std::max((max_len + P.bs - 1) / P.bs - P.tail, 0);   // in tail mode the last block is the tail CTAs'
  const long long tiles = (long long)batch * P.Hkv * ((xmax + P.scan_tile - 1) / P.scan_tile);
  long long grid = c->sm_count - tail_ctas(c, batch);
  if (grid > CKV_MAX_SCAN_CTAS) grid = CKV_MAX_SCAN_CTAS;
  if (grid > tiles) grid = tiles;
  return (int)(grid < 1 ? 1 : grid);
}

// Tail mode pays when the scan is long enough to hide the tail CTAs.  A tail warp's work is a chain of dependent
// cache misses behind the scan's traffic plus a few thousand instructions run once by a single warp: measured from
// launch, a round of tail work ends after 15 - 20 us without a new token and after 20 - 25 us with one (45 us before
// the routine's cold instructions were trimmed), whereas the scan streams about 5 MB per microsecond.  Below that
// size the scan CTAs cover every block and the append is a launch of its own, whose warps all run at once.
bool ckv_scan_wants_tail(const ckv_ctx *c, int batch, int max_len) {
  if (batch > kMaxSeqs || c->tail_mode == CKV_TAIL_OFF) return false;   // the lengths must fit the staging array
  if (c->tail_mode == CKV_TAIL_ON) return true;
  const CkvDev &P = c->dev;
  const int units = batch * P.Hkv;
  const int one_round = (units + 7) / 8;
  const int n_tail = one_round <= 16 ? std::max(1, one_round) : std::min((units + 15) / 16, std::max(16, c->sm_count / 4));
  const int rounds = (units + 8 * n_tail - 1) / (8 * n_tail);
  const double blocks = (double)units * ((max_len + P.bs - 1) / P.bs);
  const double bytes = blocks * (P.row_elems * 2.0 + (P.vhi ? CKV_D * 2.0 : P.row_elems * 2.0) + 4.0 * P.r);   // what the scan reads
  // scan microseconds: bandwidth-bound at about 5 MB/us, or issue-bound at about 6000 blocks/us (bf16 summaries).
  // A round of tail work with a new token ends 20 - 25 us after launch; measured crossover at 128K, 8 KV heads: three
  // sequences (scan about 30 us) gain a microsecond from tail mode, two (about 20 us) lose four.
  const double scan_us = std::max(bytes / 5.0e6, blocks / 6.0e3);
  return scan_us >= 30.0 * rounds;
}

cudaError_t ckv_launch_scan(ckv_ctx *c, const void *q, const int *seq_lens, int batch, int max_len,
                            const CkvNewToken *fresh_in, int *grid_out, cudaStream_t st) {
  const CkvDev &P = c->dev;
  const int units = batch * P.Hkv;
  const int n_scan = ckv_scan_grid(c, batch, max_len), n_tail = tail_ctas(c, batch);
  const int grid = n_tail + n_scan;
  CkvNewToken fresh = {};
  if (fresh_in != nullptr) {
    if (!P.tail || batch > kMaxSeqs) return cudaErrorInvalidValue;   // the new token is the tail CTAs' job
    fresh = *fresh_in;
  }
  *grid_out = n_scan;
  c->launches++;
  switch (P.G) {
    case 1: return launch_g<1>(c, q, seq_lens, units, grid, fresh, n_tail, st);
    case 2: return launch_g<2>(c, q, seq_lens, units, grid, fresh, n_tail, st);
    case 4: return launch_g<4>(c, q, seq_lens, units, grid, fresh, n_tail, st);
    case 8: return launch_g<8>(c, q, seq_lens, units, grid, fresh, n_tail, st);
  }
  return cudaErrorInvalidValue;
}
