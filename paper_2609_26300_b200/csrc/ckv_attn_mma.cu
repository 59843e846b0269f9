// Exact attention over a list of cache pages on tensor cores (bf16 layout), split along the list, with the
// removal of the selected blocks' mean-compensation terms and the final merge (Eq. 12) in the same launch.
//
// Sparse mode: the page list of a unit is the pages of its selected blocks, in position order.
// Dense mode: every page of the sequence (Eq. 12 with S = all blocks; Sec. 3.1).
//
// A CTA takes a contiguous slice of the list; each of its W warps takes every W-th page.  A warp copies its
// page (16 tokens: a 4 KB K tile and a 4 KB V tile, each contiguous in the paged pool) into one of its two
// shared-memory buffers with 16-byte cp.async pieces whose destinations are XOR-swizzled by the token row, so
// that the matrix loads below are conflict-free; rows past the sequence end are zero-filled; the next page is
// in flight while the current one is multiplied.  Then, with the G heads as the M dimension (rows 0..7 of 16)
// of mma.sync.m16n8k16:
//   S^T = Q K^T      heads x 16 tokens, Q fragments held in registers for the whole kernel
//   P   = 2^(S^T - m) per warp, running maximum raised only when exceeded by a slack; split into bf16 hi + lo
//   O  += P V        heads x 128 coordinates; the accumulator layout of S^T is the A-operand layout of P V
// For every selected block the scan kernel has already added the block's mean term |b| e^{zbar} vbar_b to
// the all-block compensation sum; here the same terms are subtracted, three blocks at a time, with one more
// P V-shaped product whose non-zero rows are the blocks' mean values (read as their stored hi + lo halves):
//   merge = exact(S) + mean(all) - mean(S) = exact(S) + mean(not S).
//
// Merge.  The scan's partials of the unit (one per scan CTA and consumer warp) exist before this kernel
// starts, so the unit's active CTAs share them out, fetch their share while their last page is in flight and
// fold it into their own partial.  What is left is one partial (m, l, acc[128]) per head and CTA:
//   * sparse mode launches the unit's splits (at most 8) as one thread-block cluster: every CTA stores its
//     partial of head g into the shared memory of CTA g mod cluster size (distributed-shared-memory stores), and
//     after one cluster barrier that CTA reduces the head from its own shared memory and writes the output row
//     and the log-sum-exp.  Nobody's shared memory is read remotely, so no CTA waits for another before it
//     leaves (the pull version, remote loads between two barriers, was 3 us slower per step);
//   * dense mode (more splits than a cluster holds), and sparse mode when a cluster cannot be placed, publish the
//     partials in global memory and bump the unit's counter; the CTA that finds the counter complete reads them
//     back and writes the output.  The counter is left at zero for the next step.
#include <mutex>

#include "ckv_internal.cuh"
#include "ckv_mma.cuh"
#include "ckv_cluster.cuh"

namespace {

constexpr int kTileBytes = CKV_PAGE * CKV_D * 2;      // one head's K (or V) page in bf16: 4 KB
constexpr int kPageBytes = 2 * kTileBytes;            // K tile | V tile
constexpr int kRowBytes = CKV_D * 2;                  // 256
constexpr int kMeanSlots = 4;                         // mean-value rows (512 B each) a warp can hold
constexpr int kMeanFlush = 3;                         // ... of which at most 3 wait for removal while one is in flight
constexpr int kZeroRow = kMeanSlots * 512;            // offset of the row of zeros inside the aux area
constexpr int kLsOff = kZeroRow + 256;                // then log2 of the blocks' mean-compensation weights: [slot][G] float
constexpr int kAuxBytes = kLsOff + 256;
constexpr int kMaxEntries = 32;                       // partials a CTA folds per round: one per lane
constexpr int kPartBytes = CKV_PART_STRIDE * 4;       // one head's partial

template <int W> constexpr size_t dyn_smem() { return (size_t)W * (2 * kPageBytes + kAuxBytes); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  // valid == false copies nothing and zero-fills the 16 bytes
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kMaxCluster = 8;    // splits of a unit that can be one cluster (the portable size; 13 measured far slower)

// RM: the mean terms of the selected blocks are removed with the stored mean-value rows (bf16 summaries); otherwise
// through the tokens' weights, and the row machinery is not compiled in.
template <int G, bool DENSE, int W, bool CL, bool RM>
__global__ void __launch_bounds__(W * 32, DENSE ? 1 : 2)
ckv_attn_mma_kernel(CkvDev P, const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_pool,
                    const __nv_bfloat16 *__restrict__ v_pool, const int *__restrict__ page_table,
                    const int *__restrict__ seq_lens, const int *__restrict__ sel_ids,
                    const int *__restrict__ sel_cnt, int kcap, int pages_per_split, int scan_grid, int units,
                    __nv_bfloat16 *__restrict__ out, float *__restrict__ lse) {
  extern __shared__ __align__(128) unsigned char smem[];   // [W warps][2 buffers][K tile | V tile], then [W warps][aux]
  __shared__ float s_M[G], s_den[G];
  __shared__ int s_last;
  // Cluster merge: where the other splits of the unit deposit their partials of the heads this CTA reduces.
  // Entry (j * cluster size + source rank) belongs to head (this rank + j * cluster size).
  __shared__ __align__(16) float s_recv[CL ? (G + kMaxCluster) * CKV_PART_STRIDE : 4];
  if (CL) cluster_arrive_relaxed();   // first phase of the cluster barrier: "this CTA runs, its shared memory exists"

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int head = lane >> 2, qd = lane & 3;
  const bool hv = head < G;
  const int unit = blockIdx.y, s = ckv_div_hkv(P, unit), h = unit - s * P.Hkv;
  const int pshift = P.ppb == 1 ? 0 : (P.ppb == 2 ? 1 : 2);
  const int p0 = blockIdx.x * pages_per_split;

  // ---- first round trip: everything that depends on nothing else is requested together ----
  const int n_raw = seq_lens[s];
  const int cnt_raw = DENSE ? 0 : sel_cnt[unit];
  int blk0 = -1;   // block of the page this lane will look up first (read before the list length is known)
  if (!DENSE) {
    const int i = p0 + warp + W * lane;
    if (i < kcap * P.ppb) blk0 = sel_ids[(size_t)unit * kcap + (i >> pshift)];
  }
  const int N = max(min(n_raw, P.max_blocks * P.bs), 0);
  const int X = (N + P.bs - 1) >> P.lg_bs;
  const int nsel = DENSE ? X : min(cnt_raw, kcap);
  const int total = DENSE ? (N + CKV_PAGE - 1) / CKV_PAGE : nsel * P.ppb;
  const bool comp = !DENSE && nsel < X && !(P.variant & CKV_VARIANT_DROP);
  const int p1 = min(p0 + pages_per_split, total);
  float *part = P.attn_part + ((size_t)unit * CKV_MAX_SPLITS + blockIdx.x) * G * CKV_PART_STRIDE;
  // Cluster merge: CTA r of the cluster (= split r of the unit) reduces heads r, r + cluster size, ...  Every CTA
  // stores its partial of a head into the shared memory of the CTA that reduces it; one cluster barrier later the
  // data is local there.  No CTA's shared memory is read remotely, so nobody has to wait before leaving.
  // `num` holds this CTA's numerators (thread t: element t, t + W * 32, ... of [G][CKV_D]); `have` is false for a
  // split without pages, which only announces an empty partial.
  auto cluster_merge = [&](const float *num, bool have) {
    cluster_wait();   // every CTA of the cluster has started
    const uint32_t rank = cluster_rank(), csize = cluster_size();
    const uint32_t recv0 = (uint32_t)__cvta_generic_to_shared(s_recv);
    // g / csize for a head index g < 8, by counting (a division by the run-time cluster size is two dozen instructions,
    // at the very end of the kernel's dependent chain)
    auto div_c = [&](uint32_t g) { uint32_t qd_ = 0; for (uint32_t m = csize; m <= g; m += csize) ++qd_; return qd_; };
    constexpr int NP = (G * CKV_D + W * 32 - 1) / (W * 32);
    if (have) {
#pragma unroll
      for (int it = 0; it < NP; ++it) {
        const int idx = tid + it * W * 32;
        if (idx < G * CKV_D) {
          const uint32_t g = idx / CKV_D, c = idx % CKV_D;
          const uint32_t gq = div_c(g) * csize;
          const uint32_t ent = gq + rank;
          st_cluster_f32(cluster_map(recv0 + (ent * CKV_PART_STRIDE + 4 + c) * 4, g - gq), num[it]);
        }
      }
    }
    if (tid < G) {
      const uint32_t gq = div_c((uint32_t)tid) * csize;
      const uint32_t ent = gq + rank;
      st_cluster_f32x2(cluster_map(recv0 + ent * kPartBytes, (uint32_t)tid - gq),
                       have ? s_M[tid] : -CUDART_INF_F, have ? s_den[tid] : 0.f);
    }
    cluster_sync_all();   // release the stores, acquire everybody else's
    for (int g = (int)rank, j = 0; g < G; g += (int)csize, ++j) {
      const float *e0 = s_recv + (size_t)j * csize * CKV_PART_STRIDE;
      float2 ml = make_float2(-CUDART_INF_F, 0.f);
      if (lane < (int)csize) ml = *reinterpret_cast<const float2 *>(e0 + lane * CKV_PART_STRIDE);
      const float M = warp_max(ml.x);
      const float sc = exp2_diff(ml.x, M);
      const float den = warp_sum(ml.y * sc);
      for (int c = tid; c < CKV_D; c += W * 32) {
        float o = 0.f;
#pragma unroll
        for (int e = 0; e < kMaxCluster; ++e) {
          const float sce = __shfl_sync(0xffffffffu, sc, e);
          if (e < (int)csize && sce != 0.f) o = fmaf(e0[e * CKV_PART_STRIDE + 4 + c], sce, o);
        }
        out[((size_t)s * P.Hq + h * G + g) * CKV_D + c] = __float2bfloat16_rn(o / den);
      }
      if (lse != nullptr && tid == 0) lse[(size_t)s * P.Hq + h * G + g] = (M + log2f(den)) * kLn2;
    }
  };
  if (p0 >= total) {   // no pages for this split
    if (total == 0) {    // an empty unit (the same for every split of it): its output is defined as zero
      if (blockIdx.x == 0) {
        for (int idx = tid; idx < G * CKV_D; idx += W * 32)
          out[((size_t)s * P.Hq + h * G) * CKV_D + idx] = __float2bfloat16_rn(0.f);
        if (lse != nullptr && tid < G) lse[(size_t)s * P.Hq + h * G + tid] = -CUDART_INF_F;
      }
      return;
    }
    if (CL) cluster_merge(nullptr, false);   // it still takes part in the cluster's merge, with an empty partial
    return;
  }
  const int n_active = (int)ckv_udiv24((unsigned)(total + pages_per_split - 1), (unsigned)pages_per_split);   // splits of this unit that have pages

  unsigned char *wtiles = smem + (size_t)warp * 2 * kPageBytes;
  const uint32_t wtiles_u32 = (uint32_t)__cvta_generic_to_shared(wtiles);
  unsigned char *waux = smem + (size_t)W * 2 * kPageBytes + (size_t)warp * kAuxBytes;
  const uint32_t aux_u32 = (uint32_t)__cvta_generic_to_shared(waux);
  // the row of zeros every unused row of the mean-value product points at
  if (lane < 16) reinterpret_cast<uint4 *>(waux + kZeroRow)[lane] = make_uint4(0u, 0u, 0u, 0u);

  const float sl2 = P.scale * kLog2e;
  float acc[16][2];
#pragma unroll
  for (int t = 0; t < 16; ++t) { acc[t][0] = 0.f; acc[t][1] = 0.f; }
  float m_ref = -CUDART_INF_F, l_acc = 0.f;
  const int *pt_row = page_table + (size_t)s * P.max_pages_per_seq;
  const int n_mine = max((p1 - p0 - warp + W - 1) / W, 0);   // this warp's pages: list index p0 + warp + W n
  const float *lz = P.lz + (size_t)unit * P.max_blocks * G;
  const __nv_bfloat16 *vmean = P.vmean + (size_t)unit * P.max_blocks * P.row_elems;
  const bool mean_lo = P.row_elems == CKV_ROW_ELEMS;   // the mean-value rows carry lo halves (fp32-precision summaries)
  // How a selected block's mean term |b| e^{zbar} vbar_b (part of the scan's all-block sum) is taken out again.
  // vbar_b is the mean of the block's value rows, so with full-precision summaries it is enough to lower the weight
  // of each of the block's tokens by e^{zbar}: sum_j (p_j - e^{zbar}) v_j = sum_j p_j v_j - |b| e^{zbar} vbar_b up to
  // the 2^-18 rounding of the stored row, with no row to fetch and no extra product.  bf16 summaries round vbar to
  // 2^-9, which would leave a visible remainder: they keep the product with the stored rows (remove_means).
  const bool tok_rm = !RM && comp, row_rm = RM && comp;
  const float lg_bs = log2f((float)P.bs), lg_last = log2f((float)max(N - (X - 1) * P.bs, 1));
  bool bad = false;

  // the scan partials this CTA folds in: partial j of the unit goes to split j % n_active
  constexpr int kSlotsPerWarp = (kPageBytes / (G * kPartBytes)) < ((kMaxEntries - W) / W) ? (kPageBytes / (G * kPartBytes))
                                                                                       : ((kMaxEntries - W) / W);
  constexpr int kSlots = W * kSlotsPerWarp;
  int my_cnt = 0;               // scan partials this CTA folds in; known once the scan slots are (below)
  const float *cp0 = nullptr;
  const size_t step = (size_t)G * CKV_PART_STRIDE;
  // start the copies of this warp's share of the round that begins at `base` into its buffer `bufsel`
  auto issue_comp = [&](int bufsel, int base) {
#pragma unroll
    for (int k = 0; k < kSlotsPerWarp; ++k) {
      const int idx = base + warp * kSlotsPerWarp + k;
      if (idx < my_cnt) {
        const float *src = cp0 + (size_t)(blockIdx.x + (size_t)idx * n_active) * step;
        const uint32_t dst = wtiles_u32 + bufsel * kPageBytes + k * (G * kPartBytes);
        for (int c = lane; c < G * (kPartBytes / 16); c += 32) cp_async16(dst + 16 * c, src + 4 * c, true);
      }
    }
  };

  struct PageRef { int phys, ntok, blk; bool first; };
  auto resolve = [&](int i, int blk) {   // list index -> physical page; blk is the selected block (sparse mode)
    PageRef r{-1, 0, -1, false};
    int page = i;
    bool ok = true;
    if (!DENSE) {
      ok = blk >= 0 && blk < X;
      r.blk = ok ? blk : -1;
      page = (r.blk << pshift) + (i & (P.ppb - 1));
      r.first = ok && (i & (P.ppb - 1)) == 0;
    }
    if (ok) {
      r.ntok = min(CKV_PAGE, N - page * CKV_PAGE);
      if (r.ntok > 0) {
        r.phys = pt_row[page];
        if (r.phys < 0 || r.phys >= P.num_pages) { r.phys = -1; bad = true; }
      } else {
        r.ntok = 0;
      }
    }
    return r;
  };
  // Page lookups are dependent loads; lane l does the lookup of page (chunk base + l) so that a chunk of 32 pages
  // costs one round trip, and fetch(n), called once per page in increasing order, hands the result to all lanes.
  PageRef mine{-1, 0, -1, false};
  auto fetch = [&](int n) {
    if ((n & 31) == 0) {
      mine = PageRef{-1, 0, -1, false};
      if (n + lane < n_mine) {
        const int i = p0 + warp + W * (n + lane);
        int blk = -1;
        if (!DENSE) blk = n == 0 ? blk0 : sel_ids[(size_t)unit * kcap + (i >> pshift)];
        mine = resolve(i, blk);
      }
    }
    PageRef r;
    r.phys = __shfl_sync(0xffffffffu, mine.phys, n & 31);
    r.ntok = __shfl_sync(0xffffffffu, mine.ntok, n & 31);
    r.blk = __shfl_sync(0xffffffffu, mine.blk, n & 31);
    r.first = __shfl_sync(0xffffffffu, (int)mine.first, n & 31) != 0;
    return r;
  };
  // start the copies of one page into buffer `buf`: 256 16-byte pieces per tile, 8 per lane; piece c of row r
  // lands at chunk c ^ (r & 7) of the row; the block's mean-value row goes to aux slot `slot`
  auto issue = [&](const PageRef &r, int buf, int slot) {
    if (r.phys >= 0) {
      const size_t src = ((size_t)r.phys * P.Hkv + h) * (CKV_PAGE * CKV_D);
      const uint32_t kb = wtiles_u32 + buf * kPageBytes;
      const uint32_t vb = kb + kTileBytes;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int idx = lane + 32 * k, row = idx >> 4, c = idx & 15;
        const uint32_t off = (uint32_t)(row * kRowBytes + ((c ^ (row & 7)) << 4));
        const bool valid = row < r.ntok;
        const size_t so = src + (size_t)(valid ? row : 0) * CKV_D + 8 * c;
        cp_async16(kb + off, k_pool + so, valid);
        cp_async16(vb + off, v_pool + so, valid);
      }
      if (row_rm && r.first) {   // verbatim: hi halves then lo halves, swizzled by block index
        if (mean_lo || lane < 16)
          cp_async16(aux_u32 + 512 * slot + 16 * lane, vmean + (size_t)r.blk * P.row_elems + 8 * lane, true);
        if (lane < G)          // and log2 of the weight of its mean term, for every head
          cp_async4(aux_u32 + kLsOff + (slot * G + lane) * 4, lz + (size_t)lane * P.max_blocks + r.blk);
      }
      if (tok_rm && lane < G)  // log2 of the block's mean-term weight, per head, beside the page's buffer
        cp_async4(aux_u32 + kLsOff + (buf * G + lane) * 4, lz + (size_t)lane * P.max_blocks + r.blk);
    }
  };

  // Blocks whose mean term |b| e^{zbar} vbar_b is still to be taken back out (it is part of the all-block sum the
  // scan produced): up to kMeanFlush of them are removed by one product, weights x mean-value rows.
  int bb[kMeanFlush], bsl[kMeanFlush], nb = 0;
#pragma unroll
  for (int j = 0; j < kMeanFlush; ++j) { bb[j] = 0; bsl[j] = 0; }
  auto remove_means = [&]() {
    float zl[2] = {-CUDART_INF_F, -CUDART_INF_F};
    if (hv && qd < 2) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int j = 2 * qd + e;
        if (j < nb) {
          const int slot = j == 0 ? bsl[0] : (j == 1 ? bsl[1] : bsl[2]);
          zl[e] = *reinterpret_cast<const float *>(waux + kLsOff + (slot * G + head) * 4);
        }
      }
    }
    float zmax = fmaxf(zl[0], zl[1]);
    zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 1));
    zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 2));
    if (zmax > m_ref + CKV_RESCALE_SLACK) {
      const float sc = exp2_diff(m_ref, zmax);
      m_ref = zmax;
      l_acc *= sc;
#pragma unroll
      for (int t = 0; t < 16; ++t) { acc[t][0] *= sc; acc[t][1] *= sc; }
    }
    const float w0 = zl[0] == -CUDART_INF_F ? 0.f : fast_exp2(zl[0] - m_ref);
    const float w1 = zl[1] == -CUDART_INF_F ? 0.f : fast_exp2(zl[1] - m_ref);
    l_acc -= w0 + w1;
    // A operand: columns 0..nb-1 (the real rows of the B operand) hold the negated weights
    const uint32_t wh = pack_bf16(-w0, -w1);
    const uint32_t wl = pack_bf16(-(w0 - bf16_round(w0)), -(w1 - bf16_round(w1)));
    // B operand: row j < nb is the mean-value row of batch entry j, every other row the row of zeros
    const int r = ((lane >> 3) & 1) * 8 + (lane & 7);
    const bool real = r < nb;
    const int rblk = r == 0 ? bb[0] : (r == 1 ? bb[1] : bb[2]);
    const int rslot = r == 0 ? bsl[0] : (r == 1 ? bsl[1] : bsl[2]);
    const uint32_t rowaddr = aux_u32 + 512 * (real ? rslot : 0);
    const int cpar = lane >> 4;
#pragma unroll
    for (int t2 = 0; t2 < 8; ++t2) {
      const uint32_t coff = (uint32_t)(swz_chunk(2 * t2 + cpar, rblk) << 4);
      uint32_t vh[4], vl[4];
      ldmatrix_x4_trans(vh, real ? rowaddr + coff : aux_u32 + kZeroRow);
      ldmatrix_x4_trans(vl, real && mean_lo ? rowaddr + 256 + coff : aux_u32 + kZeroRow);   // no lo halves: zeros
      mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh, 0u, vh[0], vh[1]);
      mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wl, 0u, vh[0], vh[1]);
      mma_rows8(acc[2 * t2][0], acc[2 * t2][1], wh, 0u, vl[0], vl[1]);
      mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh, 0u, vh[2], vh[3]);
      mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wl, 0u, vh[2], vh[3]);
      mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], wh, 0u, vl[2], vl[3]);
    }
    nb = 0;
  };

  // Mean-value slots are handed out in ring order when a block's first page is issued.  At most kMeanFlush
  // recorded blocks, the page being multiplied and the page in flight hold a slot at any time: <= kMeanSlots.
  int si = 0;
  auto take_slot = [&](const PageRef &r) {
    const int slot = si;
    if (row_rm && r.first && r.phys >= 0) si = (si + 1) & (kMeanSlots - 1);
    return slot;
  };
  PageRef cur{-1, 0, -1, false};
  int cur_slot = 0;
  if (n_mine > 0) {
    cur = fetch(0);
    cur_slot = take_slot(cur);
    issue(cur, 0, cur_slot);
  }
  // Everything the first page copy does not need is requested behind it: the queries (first used by the first
  // product) and the place of the unit's scan partials (first used with the last page).
  // Q fragments: A operand rows 0..7 = heads, scaled logits come out of the products in log2 units
  uint32_t qa[8][2];
  {
    const __nv_bfloat16 *qrow = q + ((size_t)s * P.Hq + h * G + (hv ? head : 0)) * CKV_D;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        // rows G..7 repeat head 0: finite values whose products are never used (their weights are zero), and a
        // load that nothing has to look at before the first product
        qa[ks][hh] = __ldg(reinterpret_cast<const uint32_t *>(qrow + 16 * ks + 8 * hh + 2 * qd));
      }
  }
  if (comp) {
    int efirst = 0, n_comp = 0;   // where the unit's scan partials sit
    unit_scan_entries(P, CkvClampedLens{seq_lens, P.max_blocks * P.bs}, units, unit, scan_grid, lane, efirst, n_comp);
    my_cnt = n_comp > (int)blockIdx.x ? (int)ckv_udiv24((unsigned)(n_comp - (int)blockIdx.x + n_active - 1), (unsigned)n_active) : 0;
    cp0 = P.comp_part + (size_t)efirst * G * CKV_PART_STRIDE;
  }

  if (n_mine == 0) issue_comp(1, 0);   // a warp without pages only brings in its share of the scan partials
  cp_async_commit();
  for (int n = 0, buf = 0; n < n_mine; ++n, buf ^= 1) {
    PageRef nxt{-1, 0, -1, false};
    int nxt_slot = 0;
    if (n + 1 < n_mine) {
      nxt = fetch(n + 1);
      nxt_slot = take_slot(nxt);
      issue(nxt, buf ^ 1, nxt_slot);
    } else {
      issue_comp(buf ^ 1, 0);   // the other buffer is idle during the last page
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncwarp();
    if (cur.phys >= 0) {
      const uint32_t kb = wtiles_u32 + buf * kPageBytes;
      const uint32_t vb = kb + kTileBytes;
      // ---- S^T = Q K^T: heads x 16 tokens (two n-tiles of 8 tokens) ----
      float sv[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, sv2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
      {
        const int lrow = lane & 7, lmat = lane >> 3;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int r = nt * 8 + lrow;
          const uint32_t rowaddr = kb + r * kRowBytes;
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // two 16-coordinate steps per ldmatrix.x4
            uint32_t b[4];
            ldmatrix_x4(b, rowaddr + (uint32_t)(((4 * j + lmat) ^ (r & 7)) << 4));
            mma_rows8(sv[nt][0], sv[nt][1], qa[2 * j][0], qa[2 * j][1], b[0], b[1]);
            mma_rows8(sv2[nt][0], sv2[nt][1], qa[2 * j + 1][0], qa[2 * j + 1][1], b[2], b[3]);
          }
          sv[nt][0] += sv2[nt][0]; sv[nt][1] += sv2[nt][1];
        }
      }
      // ---- softmax weights for this thread's head and its four tokens ----
      float tmax = -CUDART_INF_F;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool ok = hv && nt * 8 + 2 * qd + e < cur.ntok;
          sv[nt][e] = ok ? sv[nt][e] * sl2 : -CUDART_INF_F;
          tmax = fmaxf(tmax, sv[nt][e]);
        }
      // log2 of e^{zbar} of the page's block for this lane's head (token-weight removal)
      float lzt = -CUDART_INF_F;
      if (tok_rm && hv)
        lzt = *reinterpret_cast<const float *>(waux + kLsOff + (buf * G + head) * 4) - (cur.blk == X - 1 ? lg_last : lg_bs);
      tmax = fmaxf(tmax, lzt);
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
      if (tmax > m_ref + CKV_RESCALE_SLACK) {
        const float sc = exp2_diff(m_ref, tmax);
        m_ref = tmax;
        l_acc *= sc;
#pragma unroll
        for (int t = 0; t < 16; ++t) { acc[t][0] *= sc; acc[t][1] *= sc; }
      }
      const float wtok = lzt == -CUDART_INF_F ? 0.f : fast_exp2(lzt - m_ref);
      uint32_t ph[2], pl[2];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float p[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          p[e] = sv[nt][e] == -CUDART_INF_F ? 0.f : fast_exp2(sv[nt][e] - m_ref) - wtok;
          l_acc += p[e];
        }
        ph[nt] = pack_bf16(p[0], p[1]);
        pl[nt] = pack_bf16(p[0] - bf16_round(p[0]), p[1] - bf16_round(p[1]));
      }
      // ---- O += P V ----
      {
        const int r = ((lane >> 3) & 1) * 8 + (lane & 7);
        const uint32_t rowaddr = vb + r * kRowBytes;
        const int cpar = lane >> 4;
#pragma unroll
        for (int t2 = 0; t2 < 8; ++t2) {   // two 8-coordinate n-tiles per ldmatrix.x4
          uint32_t v[4];
          ldmatrix_x4_trans(v, rowaddr + (uint32_t)(((2 * t2 + cpar) ^ (r & 7)) << 4));
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], ph[0], ph[1], v[0], v[1]);
          mma_rows8(acc[2 * t2][0], acc[2 * t2][1], pl[0], pl[1], v[0], v[1]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], ph[0], ph[1], v[2], v[3]);
          mma_rows8(acc[2 * t2 + 1][0], acc[2 * t2 + 1][1], pl[0], pl[1], v[2], v[3]);
        }
      }
      if (row_rm && cur.first) {   // its mean-value row sits in aux slot cur_slot
#pragma unroll
        for (int j = 0; j < kMeanFlush; ++j)
          if (j == nb) { bb[j] = cur.blk; bsl[j] = cur_slot; }
        ++nb;
      }
    }
    if constexpr (RM) {
      if (nb == kMeanFlush || (nb > 0 && n + 1 == n_mine)) remove_means();
    }
    __syncwarp();   // the page buffer (and, after a removal, the mean-value slots) may be overwritten from here on
    cur = nxt;
    cur_slot = nxt_slot;
  }
  cp_async_wait<0>();
  __syncwarp();
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(P.status, CKV_DEV_BAD_PAGE);

  // ---- CTA partial: fold the warps (each with its own running maximum) and this CTA's scan partials ----
  // A warp's partial [G][CKV_PART_STRIDE] goes into the buffer of its last page; the other buffer holds its
  // share of the scan partials.  Entry e < W is warp e's partial, entry W + c is scan-partial slot c.
  auto red_buf = [&](int e) {
    const int nm = max((p1 - p0 - e + W - 1) / W, 0);
    return nm > 0 ? (nm - 1) & 1 : 0;
  };
  auto region = [&](int e, int b) { return (int)(((size_t)e * 2 * kPageBytes + (size_t)b * kPageBytes) / 4); };   // in floats
  float *sf = reinterpret_cast<float *>(smem);
  // scale factors [entry][G] and entry offsets live in the aux area, which the page loop no longer needs
  float(*s_scale)[G] = reinterpret_cast<float(*)[G]>(smem + (size_t)W * 2 * kPageBytes);
  int *s_ent = reinterpret_cast<int *>(smem + (size_t)W * 2 * kPageBytes + kMaxEntries * G * 4);
  __syncthreads();   // every warp is done with its aux rows
  l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 1);
  l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 2);
  if (hv) {
    float *r = sf + region(warp, red_buf(warp)) + head * CKV_PART_STRIDE;
#pragma unroll
    for (int t = 0; t < 16; ++t) *reinterpret_cast<float2 *>(r + 4 + 8 * t + 2 * qd) = make_float2(acc[t][0], acc[t][1]);
    if (qd == 0) { r[0] = m_ref; r[1] = l_acc; }
  }
  if (tid < W + kSlots) {
    int off;
    if (tid < W) {
      off = region(tid, red_buf(tid));
    } else {
      const int c = tid - W, we = c / kSlotsPerWarp, k = c % kSlotsPerWarp;
      off = region(we, red_buf(we) ^ 1) + k * G * CKV_PART_STRIDE;
    }
    s_ent[tid] = off;
  }
  constexpr int NI = (G * CKV_D + W * 32 - 1) / (W * 32);
  float num[NI];
  for (int base = 0;; base += kSlots) {
    __syncthreads();   // the entries of this round are in place
    for (int g = warp; g < G; g += W) {   // per head: maximum, scale factor of every entry, normaliser
      const bool valid = lane < W ? (base == 0 || lane == 0) : (lane < W + kSlots && base + lane - W < my_cnt);
      const float *p = sf + s_ent[lane < W + kSlots ? lane : 0] + g * CKV_PART_STRIDE;
      const float m = valid ? p[0] : -CUDART_INF_F, l = valid ? p[1] : 0.f;
      const float M = warp_max(m);
      const float sc = exp2_diff(m, M);
      const float den = warp_sum(l * sc);
      s_scale[lane][g] = sc;
      if (lane == 0) { s_M[g] = M; s_den[g] = den; }
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < NI; ++it) num[it] = 0.f;
    // every entry is read (a slot that holds nothing is multiplied by a zero that replaces its value, not by
    // its bits), so the loads of all entries are independent and in flight together
#pragma unroll 4
    for (int e = 0; e < W + kSlots; ++e) {
      const float *ep = sf + s_ent[e] + 4;
#pragma unroll
      for (int it = 0; it < NI; ++it) {
        const int idx = min(tid + it * W * 32, G * CKV_D - 1);
        const int g = idx / CKV_D, c = idx % CKV_D;
        const float sc = s_scale[e][g];
        const float x = ep[g * CKV_PART_STRIDE + c];
        num[it] = fmaf(sc != 0.f ? x : 0.f, sc, num[it]);
      }
    }
    if (base + kSlots >= my_cnt) break;
    // more scan partials than slots (few splits, many scan CTAs): keep the result as entry 0 and go round again
    __syncthreads();
    {
      float *carry = sf + s_ent[0];
#pragma unroll
      for (int it = 0; it < NI; ++it) {
        const int idx = tid + it * W * 32;
        if (idx < G * CKV_D) carry[(idx / CKV_D) * CKV_PART_STRIDE + 4 + idx % CKV_D] = num[it];
      }
      if (tid < G) { carry[tid * CKV_PART_STRIDE] = s_M[tid]; carry[tid * CKV_PART_STRIDE + 1] = s_den[tid]; }
    }
    issue_comp(red_buf(warp) ^ 1, base + kSlots);
    cp_async_commit();
    cp_async_wait<0>();
  }
  if constexpr (CL) {
    cluster_merge(num, true);
    return;
  } else {
#pragma unroll
  for (int it = 0; it < NI; ++it) {
    const int idx = tid + it * W * 32;
    if (idx < G * CKV_D) part[(idx / CKV_D) * CKV_PART_STRIDE + 4 + idx % CKV_D] = num[it];
  }
  if (tid < G) { part[tid * CKV_PART_STRIDE] = s_M[tid]; part[tid * CKV_PART_STRIDE + 1] = s_den[tid]; }

  // ---- the last split of the unit to finish merges the unit's partials into the output (Eq. 12) ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int done = atomicAdd(P.unit_done + unit, 1);
    s_last = done == n_active - 1;
    if (s_last) P.unit_done[unit] = 0;   // leave the counter ready for the next step
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float *ap0 = P.attn_part + (size_t)unit * CKV_MAX_SPLITS * G * CKV_PART_STRIDE;
  const int c4 = 4 * lane;
  for (int g = warp; g < G; g += W) {   // a warp per head; lane i holds (m, l) of partials i and i + 32, and four coordinates
    const float *ag = ap0 + (size_t)g * CKV_PART_STRIDE;
    float2 ml0 = make_float2(-CUDART_INF_F, 0.f), ml1 = make_float2(-CUDART_INF_F, 0.f);
    if (lane < n_active) ml0 = __ldcg(reinterpret_cast<const float2 *>(ag + (size_t)lane * step));
    if (lane + 32 < n_active) ml1 = __ldcg(reinterpret_cast<const float2 *>(ag + (size_t)(lane + 32) * step));
    float4 a[8];   // the first eight partials are requested before the scale factors are known
#pragma unroll
    for (int k = 0; k < 8; ++k)
      a[k] = k < n_active ? __ldcg(reinterpret_cast<const float4 *>(ag + (size_t)k * step + 4 + c4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    const float M = warp_max(fmaxf(ml0.x, ml1.x));
    const float sc0 = exp2_diff(ml0.x, M), sc1 = exp2_diff(ml1.x, M);
    const float den = warp_sum(ml0.y * sc0 + ml1.y * sc1);
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = 0; i < n_active; i += 8) {
      if (i > 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
          a[k] = i + k < n_active ? __ldcg(reinterpret_cast<const float4 *>(ag + (size_t)(i + k) * step + 4 + c4)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int ii = i + k;
        const float sc = __shfl_sync(0xffffffffu, ii < 32 ? sc0 : sc1, ii & 31);
        if (ii < n_active && sc != 0.f) {
          o.x = fmaf(a[k].x, sc, o.x); o.y = fmaf(a[k].y, sc, o.y);
          o.z = fmaf(a[k].z, sc, o.z); o.w = fmaf(a[k].w, sc, o.w);
        }
      }
    }
    const float inv = 1.0f / den;
    uint2 o2;
    o2.x = pack_bf16(o.x * inv, o.y * inv);
    o2.y = pack_bf16(o.z * inv, o.w * inv);
    *reinterpret_cast<uint2 *>(out + ((size_t)s * P.Hq + h * G + g) * CKV_D + c4) = o2;
    if (lse != nullptr && lane == 0) lse[(size_t)s * P.Hq + h * G + g] = (M + log2f(den)) * kLn2;
  }
  }   // !CL
}

constexpr int kSparseWarps = 4, kDenseWarps = 8;

// Whether `n_splits` sparse CTAs of this instantiation can be placed as one cluster on the current device.
template <int G>
bool cluster_fits(int n_splits, cudaStream_t st) {
  if (n_splits > kMaxCluster) return false;
  // the answer is a property of the device: cached per device (and per G: the template instantiates one table
  // each), behind a mutex, since contexts on several devices or host threads may ask at once
  constexpr int kMaxDev = 64;
  static std::mutex mtx;
  static int table[kMaxDev][kMaxCluster + 1];   // 0 unknown, 1 fits, 2 does not
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) { (void)cudaGetLastError(); return false; }
  std::lock_guard<std::mutex> lock(mtx);
  int *cache = table[dev];
  if (cache[n_splits] != 0) return cache[n_splits] == 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, 1, 1);
  cfg.blockDim = dim3(kSparseWarps * 32);
  cfg.dynamicSmemBytes = dyn_smem<kSparseWarps>();
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_splits; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, ckv_attn_mma_kernel<G, false, kSparseWarps, true, true>, &cfg);
  if (e != cudaSuccess) (void)cudaGetLastError();
  cache[n_splits] = (e == cudaSuccess && n > 0) ? 1 : 2;
  return cache[n_splits] == 1;
}

template <int G>
cudaError_t launch_g(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                     const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt, int kcap,
                     dim3 grid, int pps, int scan_grid, void *out, float *lse, cudaStream_t st) {
  const int units = (int)grid.y;
  const __nv_bfloat16 *qp = (const __nv_bfloat16 *)q, *kp = (const __nv_bfloat16 *)k_pool, *vp = (const __nv_bfloat16 *)v_pool;
  if (dense) {
    ckv_attn_mma_kernel<G, true, kDenseWarps, false, false><<<grid, kDenseWarps * 32, dyn_smem<kDenseWarps>(), st>>>(
        c->dev, qp, kp, vp, page_table, seq_lens, sel_ids, sel_cnt, kcap, pps, scan_grid, units, (__nv_bfloat16 *)out, lse);
    return cudaGetLastError();
  }
  const bool rm = c->dev.row_elems == CKV_D;   // bf16 summaries: removal with the stored mean-value rows
  if (cluster_fits<G>((int)grid.x, st)) {   // the unit's splits as one cluster: partials never leave the SMs
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kSparseWarps * 32);
    cfg.dynamicSmemBytes = dyn_smem<kSparseWarps>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = grid.x; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (rm)
      return cudaLaunchKernelEx(&cfg, ckv_attn_mma_kernel<G, false, kSparseWarps, true, true>, c->dev, qp, kp, vp, page_table,
                                seq_lens, sel_ids, sel_cnt, kcap, pps, scan_grid, units, (__nv_bfloat16 *)out, lse);
    return cudaLaunchKernelEx(&cfg, ckv_attn_mma_kernel<G, false, kSparseWarps, true, false>, c->dev, qp, kp, vp, page_table,
                              seq_lens, sel_ids, sel_cnt, kcap, pps, scan_grid, units, (__nv_bfloat16 *)out, lse);
  }
  if (rm)
    ckv_attn_mma_kernel<G, false, kSparseWarps, false, true><<<grid, kSparseWarps * 32, dyn_smem<kSparseWarps>(), st>>>(
        c->dev, qp, kp, vp, page_table, seq_lens, sel_ids, sel_cnt, kcap, pps, scan_grid, units, (__nv_bfloat16 *)out, lse);
  else
    ckv_attn_mma_kernel<G, false, kSparseWarps, false, false><<<grid, kSparseWarps * 32, dyn_smem<kSparseWarps>(), st>>>(
        c->dev, qp, kp, vp, page_table, seq_lens, sel_ids, sel_cnt, kcap, pps, scan_grid, units, (__nv_bfloat16 *)out, lse);
  return cudaGetLastError();
}

template <int G>
cudaError_t configure_g() {
  cudaError_t e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, true, kDenseWarps, false, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_smem<kDenseWarps>());
  const int sm = (int)dyn_smem<kSparseWarps>();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, false, kSparseWarps, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, false, kSparseWarps, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, false, kSparseWarps, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ckv_attn_mma_kernel<G, false, kSparseWarps, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  return e;
}

}  // namespace

cudaError_t ckv_configure_attn_mma(const ckv_ctx *c) {
  switch (c->dev.G) {
    case 1: return configure_g<1>();
    case 2: return configure_g<2>();
    case 4: return configure_g<4>();
    case 8: return configure_g<8>();
  }
  return cudaErrorInvalidValue;
}

cudaError_t ckv_launch_attn_mma(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                                const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt,
                                int kcap, dim3 grid, int pps, int scan_grid, void *out, float *lse, cudaStream_t st) {
  switch (c->dev.G) {
    case 1: return launch_g<1>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, scan_grid, out, lse, st);
    case 2: return launch_g<2>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, scan_grid, out, lse, st);
    case 4: return launch_g<4>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, scan_grid, out, lse, st);
    case 8: return launch_g<8>(c, dense, q, k_pool, v_pool, page_table, seq_lens, sel_ids, sel_cnt, kcap, grid, pps, scan_grid, out, lse, st);
  }
  return cudaErrorInvalidValue;
}
