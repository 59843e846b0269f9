// Internal declarations shared by the CompKV CUDA translation units (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/compkv.h"

#define CKV_D 128             // head dimension the kernels are written for
#define CKV_PAGE 16           // tokens per page
#define CKV_ROW_ELEMS 256     // bf16 elements of one mean-key / mean-value summary row (128 hi halves + 128 lo halves)
#define CKV_PART_STRIDE 132   // floats per split partial: m, l, pad, pad, acc[128]
#define CKV_SCAN_TILE 32      // blocks per scan tile (rows of 512 bytes: two 16 KB bulk copies and the variances per tile)
#define CKV_SCAN_TILE_HS 64   // ... with bf16 summaries (rows of 256 bytes): the same bytes per copy.  An SM's copy engine
                              // takes about 3.8 bulk copies per microsecond whatever their size (measured), so halving
                              // the rows without doubling the tile left the scan exactly as slow as before
#define CKV_SCAN_WARPS 7       // consumer warps of a scan CTA (plus one producer warp: 256 threads), each with a partial of its own
#define CKV_MAX_SCAN_CTAS 160 // persistent scan grid is capped at this many CTAs
#define CKV_MAX_SPLITS 64     // attention partials per unit
#define CKV_RESCALE_SLACK 16.0f  // log2 units: running maxima are only raised when exceeded by this much

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Everything a kernel needs to find its data; passed by value.
struct CkvDev {
  int Hq, Hkv, G, bs, ppb, r, glayout;
  int max_blocks, max_pages_per_seq, num_pages, sink, recent;
  float scale;
  // block summaries (caller's stats buffer): mean keys / mean values as split-bf16 rows (see store_split8), variances fp32
  __nv_bfloat16 *kmean, *vmean;   // [unit][max_blocks][CKV_ROW_ELEMS]
  float *dbar;                    // [unit][max_blocks][r]
  // workspace
  float *lu;         // [unit][G][max_blocks]  log2 of the head's score term e^{l_{g,b}} sigma_hat^2_{g,b} (selection reads it)
  float *lz;         // [unit][G][max_blocks]  log2 of the block's mean-compensation weight |b| e^{zbar_{g,b}} (attention)
  float *scores;     // [unit][max_blocks]     S_b
  float *comp_part;  // [(scan CTA + 2 unit) * CKV_SCAN_WARPS + warp][G][CKV_PART_STRIDE]  all-block mean-compensation partials (see unit_scan_entries)
  float *attn_part;  // [unit][CKV_MAX_SPLITS][G][CKV_PART_STRIDE]  exact-attention partials
  int row_elems;     // bf16 elements of one mean-key / mean-value row: CKV_ROW_ELEMS, or CKV_D when only hi halves are kept
  int variant;       // ckv_variant bits
  float half_var;    // coefficient of sigma^2 in the estimated log mass: 0.5 (Eq. 9), or 0 for the first-order mass
  int scan_tile;     // blocks per scan tile: CKV_SCAN_TILE, or CKV_SCAN_TILE_HS with bf16 summaries or vhi
  int vhi;           // 1: the decode step reads the mean values' hi halves only (the lo halves, at most 2^-8 of a value,
                     // stay in the summaries for whoever exports them): the scan copies 256 of a row's 512 bytes.  The
                     // compensation term is a weighted average over thousands of blocks and ends in a bf16 output row, so
                     // the roundings neither add up nor show (measured: the output error against the oracle is the same
                     // 0.0034 maximum with and without the lo halves)
  unsigned hkv_magic;  // floor(2^32 / Hkv) + 1: x / Hkv = umulhi(x, hkv_magic) for x < 2^32 / Hkv (ckv_div_hkv)
  int lg_bs, lg_tile;  // log2 of bs and of scan_tile (both powers of two): the kernels' prologues divide by shifting --
                       // a division by a run-time value is two dozen instructions, and a prologue's time is the fetch of its
                       // own cold instructions
  int tail;          // 1: the scan launch leaves the last block of every sequence to its tail CTAs (set per step)
  int *unit_done;    // [unit] attention splits finished this step (zero between steps); null = merge is a separate launch
  int *status;       // device status word
  uint32_t spin_limit;  // polls a bounded wait makes before it gives up (ckv_debug_set; default ckv_pipe::kSpinLimit)
  int debug;         // ckv_debug_flags (test hooks; 0 in normal use)
};

struct ckv_ctx {
  ckv_layout layout;
  CkvDev dev;
  char *work;
  size_t work_bytes;
  // host staging regions inside the workspace (ckv_step_host)
  size_t stage_q, stage_knew, stage_vnew, stage_out, stage_ids, stage_cnt;
  int64_t launches;
  int sm_count;
  int tail_mode;   // ckv_tail_mode
  CUtensorMap tm_vhi;   // vhi: the mean-values region as rows of 128 bf16 (the hi halves) 512 bytes apart, boxes of 64 rows
  volatile int *host_flag;   // pinned word ckv_step_host waits on (null: stream synchronisation instead)
  int *host_flag_dev;        // the same word as the device sees it
  int host_epoch;            // number of the last ckv_step_host call that used the word
  // ckv_step_host replays a captured graph when it is called again with the same buffers and sizes
  void *hg_exec;             // cudaGraphExec_t, or null
  const void *hg_key[10];    // the six host buffers, pools, page table, lengths array
  int hg_ints[4];            // batch, rounded length bound, budget, tail mode
  int hg_launches;           // kernel launches one replay stands for
  bool hg_key_valid, hg_disabled;
};

int ckv_record_cuda_error(cudaError_t e);   // remembers e for ckv_last_cuda_error() on this thread; returns CKV_ERR_CUDA
cudaError_t ckv_configure_kernels();   // selection kernel attributes
cudaError_t ckv_configure_scan(ckv_ctx *c);   // scan kernel attributes (and, with vhi, the tensor map of the mean values)
cudaError_t ckv_configure_attn(const ckv_ctx *c);   // attention kernel attributes
cudaError_t ckv_configure_attn_mma(const ckv_ctx *c);
cudaError_t ckv_launch_attn_mma(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                                const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt,
                                int kcap, dim3 grid, int pps, int scan_grid, void *out, float *lse, cudaStream_t st);
int ckv_scan_grid(const ckv_ctx *c, int batch, int max_len);

// ---- launchers (one per translation unit) ---------------------------------------------------------
cudaError_t ckv_launch_stats_build(ckv_ctx *c, const void *k_pool, const void *v_pool, const int *page_table,
                                   const int *seq_lens, int batch, int max_len, cudaStream_t st);
cudaError_t ckv_launch_stats_export(ckv_ctx *c, int batch, float *kmean, float *dbar, float *vmean, cudaStream_t st);
cudaError_t ckv_launch_prefill(ckv_ctx *c, void *k_pool, void *v_pool, const int *page_table, int *seq_lens,
                               const void *k_src, const void *v_src, const int *new_lens, int src_stride, int batch,
                               int max_new, cudaStream_t st);
cudaError_t ckv_launch_append(ckv_ctx *c, void *k_pool, void *v_pool, const int *page_table, int *seq_lens,
                              const void *k_new, const void *v_new, int batch, cudaStream_t st);
// The new token of a fused step (append inside the scan launch); all null for a plain decode.
struct CkvNewToken {
  void *k_pool, *v_pool;      // paged pools, written at position seq_lens[s]
  const int *page_table;
  int *seq_lens;              // read as the lengths before the append; holds the new lengths when the launch is over
  const void *k_new, *v_new;  // [batch][Hkv][128]
};
// max_len is an upper bound of the lengths the step works on (after the append, if there is one).  The launch
// follows c->dev.tail; a new token needs tail mode.
cudaError_t ckv_launch_scan(ckv_ctx *c, const void *q, const int *seq_lens, int batch, int max_len,
                            const CkvNewToken *fresh, int *grid_out, cudaStream_t st);
// Whether a step of this size should run in tail mode (the scan, select and attention launches of one step must
// agree: the caller stores the answer in c->dev.tail before launching them).
bool ckv_scan_wants_tail(const ckv_ctx *c, int batch, int max_len);
cudaError_t ckv_launch_select(ckv_ctx *c, const int *seq_lens, int batch, int kcap, int scan_grid, int *sel_ids,
                              int *sel_cnt, cudaStream_t st);
cudaError_t ckv_launch_attn(ckv_ctx *c, bool dense, const void *q, const void *k_pool, const void *v_pool,
                            const int *page_table, const int *seq_lens, const int *sel_ids, const int *sel_cnt,
                            int kcap, int batch, int max_len, int scan_grid, void *out, float *lse,
                            int *n_splits_out, bool *merged_out, cudaStream_t st);
cudaError_t ckv_launch_exact_blocks(ckv_ctx *c, const void *q, const void *k_pool, const int *page_table,
                                    const int *seq_lens, int batch, int max_len, float *logZ, float *zmean, float *zvar,
                                    cudaStream_t st);
cudaError_t ckv_launch_merge(ckv_ctx *c, bool dense, const int *seq_lens, const int *sel_cnt, int n_splits,
                             int scan_grid, int batch, void *out, float *lse, cudaStream_t st);

// ---- device helpers -----------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ void bf16x8_to_float(const uint4 &u, float (&o)[8]) {
  o[0] = __uint_as_float(u.x << 16); o[1] = __uint_as_float(u.x & 0xffff0000u);
  o[2] = __uint_as_float(u.y << 16); o[3] = __uint_as_float(u.y & 0xffff0000u);
  o[4] = __uint_as_float(u.z << 16); o[5] = __uint_as_float(u.z & 0xffff0000u);
  o[6] = __uint_as_float(u.w << 16); o[7] = __uint_as_float(u.w & 0xffff0000u);
}

// Mixed-precision adds of sm_100: the bf16 operand is widened inside the instruction (exactly), so the result has the
// bits of converting first and adding in fp32, at half the instructions.
__device__ __forceinline__ void split_b32(uint32_t u, uint16_t &lo, uint16_t &hi) {
  asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u));
}
__device__ __forceinline__ float add_f32_bf16(uint16_t a, float c) {
  float r;
  asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(r) : "h"(a), "f"(c));
  return r;
}
__device__ __forceinline__ float sub_f32_bf16(uint16_t a, float c) {   // a - c
  float r;
  asm("sub.rn.f32.bf16 %0, %1, %2;" : "=f"(r) : "h"(a), "f"(c));
  return r;
}
// acc[i] += float(u[i]) for the eight bf16 values of u
__device__ __forceinline__ void add_bf16x8(const uint4 &u, float (&acc)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint16_t lo, hi;
    split_b32(w[i], lo, hi);
    acc[2 * i] = add_f32_bf16(lo, acc[2 * i]);
    acc[2 * i + 1] = add_f32_bf16(hi, acc[2 * i + 1]);
  }
}
// d[i] = float(u[i]) - m[i]
__device__ __forceinline__ void sub_bf16x8(const uint4 &u, const float (&m)[8], float (&d)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint16_t lo, hi;
    split_b32(w[i], lo, hi);
    d[2 * i] = sub_f32_bf16(lo, m[2 * i]);
    d[2 * i + 1] = sub_f32_bf16(hi, m[2 * i + 1]);
  }
}

// Eight consecutive elements as floats.  NC = read-only (non-coherent) path; use NC = false for
// data the same kernel has just written.
template <bool NC>
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&o)[8]) {
  uint4 u;
  if (NC) u = __ldg(reinterpret_cast<const uint4 *>(p));
  else u = *reinterpret_cast<const uint4 *>(p);
  bf16x8_to_float(u, o);
}
template <bool NC>
__device__ __forceinline__ void load8(const float *p, float (&o)[8]) {
  float4 a, b;
  if (NC) { a = __ldg(reinterpret_cast<const float4 *>(p)); b = __ldg(reinterpret_cast<const float4 *>(p) + 1); }
  else { a = *reinterpret_cast<const float4 *>(p); b = *(reinterpret_cast<const float4 *>(p) + 1); }
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float *p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

// Summary rows.  A mean key / mean value entry x is stored as two bf16, hi = bf16(x) and lo = bf16(x - hi): the same
// 32 bits as an fp32, relative error at most 2^-18, and directly usable as tensor-core operands (x * y is evaluated
// as hi * y + lo * y).  A row of 128 entries is 512 bytes: sixteen 16-byte chunks of hi halves (8 coordinates each),
// then sixteen chunks of lo halves.  Inside every group of 8 chunks the chunk order is XORed with (block index & 7),
// so that a matrix load touching one chunk column of 8 consecutive rows hits 8 different bank groups.
__device__ __forceinline__ int swz_chunk(int chunk, int block) { return chunk ^ (block & 7); }

// lo_half false: only the hi halves are kept (the bf16 summary layout, rows of 256 bytes).
__device__ __forceinline__ void store_split8(__nv_bfloat16 *row, int chunk, int block, const float (&x)[8], bool lo_half = true) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {   // two values per conversion instruction; the halves come back out by shift and mask
    const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    hi[i] = *reinterpret_cast<const uint32_t *>(&h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x[2 * i] - __uint_as_float(hi[i] << 16),
                                                   x[2 * i + 1] - __uint_as_float(hi[i] & 0xffff0000u));
    lo[i] = *reinterpret_cast<const uint32_t *>(&l);
  }
  const int p = swz_chunk(chunk, block) * 8;
  *reinterpret_cast<uint4 *>(row + p) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  if (lo_half) *reinterpret_cast<uint4 *>(row + CKV_D + p) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

// The eight entries of one chunk, hi + lo (hi alone when the row has no lo halves), as floats.
// NC = false for rows the same kernel has just written.
template <bool NC = true>
__device__ __forceinline__ void load_split8(const __nv_bfloat16 *row, int chunk, int block, float (&x)[8], bool lo_half = true) {
  const int p = swz_chunk(chunk, block) * 8;
  const uint4 *ph = reinterpret_cast<const uint4 *>(row + p), *pl = reinterpret_cast<const uint4 *>(row + CKV_D + p);
  const uint4 h = NC ? __ldg(ph) : *ph;
  const uint4 l = lo_half ? (NC ? __ldg(pl) : *pl) : make_uint4(0u, 0u, 0u, 0u);
  float a[8], b[8];
  bf16x8_to_float(h, a);
  bf16x8_to_float(l, b);
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = a[i] + b[i];
}

// Coordinate group of coordinate i (App. A.4 of the paper; see ckv_layout::group_layout).
__device__ __forceinline__ int group_of(int i, int r, int glayout) {
  if (r == CKV_D) return i;
  if (glayout == 0) return i / (CKV_D / r);
  const int half = CKV_D / 2;
  const int p = i < half ? i : i - half;
  return p / (half / r);
}

// Sum-reduce NV per-lane values across the 16 lanes of a half warp, sharing the work: while more
// than KEEP values remain each step halves the count (a lane sends the half it gives up and keeps
// the other), then the remaining steps are plain butterflies.  On return v[0..KEEP) hold complete
// sums; the lane with half-warp index li owns original indices
//   [ (li >> (4 - S)) * KEEP, +KEEP ),  S = log2(NV / KEEP) halving steps (S <= 4).
template <int NV, int KEEP>
__device__ __forceinline__ void reduce16(float (&v)[NV], int li) {
  int n = NV;
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    const int mask = 8 >> step;
    if (n > KEEP) {
      const int half = n / 2;
      const bool up = (li & mask) != 0;
#pragma unroll
      for (int i = 0; i < NV / 2; ++i) {
        if (i < half) {
          const float send = up ? v[i] : v[i + half];
          const float keep = up ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
        }
      }
      n = half;
    } else {
#pragma unroll
      for (int i = 0; i < KEEP; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], mask);
    }
  }
}

// Two fp32 values in one 64-bit register pair, for the packed fp32 instructions of sm_100.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// d = a * b + c on both halves (one instruction).
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x with the hardware approximation (relative error about 2^-22; -inf gives 0).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// exp2 of a difference that may involve -inf on either side without producing NaN.
__device__ __forceinline__ float exp2_diff(float a, float b) {
  return (a == -CUDART_INF_F) ? 0.0f : exp2f(a - b);
}

// Which scan partials belong to `unit`.  The scan cuts the blocks of all units into tiles of P.scan_tile blocks;
// scan CTA c gets the tiles [c * tpc, (c + 1) * tpc) and consumer warp w stores its partial for unit u in entry
// (c + 2 u) * CKV_SCAN_WARPS + w.  The (c, u) pairs that occur form a monotone staircase, so with the factor 2 the
// group behind a unit's last CTA is free.  In tail mode (P.tail) the scan CTAs leave the LAST block of every
// sequence (the one a new token lands in) to the launch's tail CTAs, whose partial takes the first entry of that
// free group.  Either way a unit's entries are contiguous: `first`, and `count` of them (zero for an empty sequence).
// len_of(i) is the clamped length of sequence i.  Must be called by all 32 lanes of a warp; every lane gets the result.
//
// The divisions of this arithmetic are done without the division instruction sequence (about 25 instructions each, and
// a kernel's prologue costs what its cold instructions cost to fetch):
// x / Hkv for unit indices (x * Hkv < 2^32, checked at creation) by a multiplication with a host-made constant;
__device__ __forceinline__ int ckv_div_hkv(const CkvDev &P, int x) {
  return P.Hkv == 1 ? x : (int)__umulhi((unsigned)x, P.hkv_magic);
}
// a / b for tile counts (a, b < 2^24, b >= 1: a step has fewer than 2^24 tiles, checked at creation) by a float
// reciprocal, exact in both operands, whose quotient is then put right by its remainder.
__device__ __forceinline__ unsigned ckv_udiv24(unsigned a, unsigned b) {
  unsigned q = (unsigned)__fdividef((float)a, (float)b);
  int r = (int)a - (int)(q * b);
  while (r < 0) { --q; r += (int)b; }
  while (r >= (int)b) { ++q; r -= (int)b; }
  return q;
}
__device__ __forceinline__ int ckv_scan_blocks(const CkvDev &P, int n) { return max(((n + P.bs - 1) >> P.lg_bs) - P.tail, 0); }   // n >= 0
template <class LenFn>
__device__ __forceinline__ void unit_scan_entries(const CkvDev &P, LenFn len_of, int units, int unit, int scan_grid,
                                                  int lane, int &first, int &count) {
  const int batch = ckv_div_hkv(P, units), s = ckv_div_hkv(P, unit), h = unit - s * P.Hkv;
  unsigned tot = 0, before = 0, mine = 0, n_mine = 0;
  for (int i = lane; i < batch; i += 32) {
    const int n = len_of(i);
    const unsigned t = (unsigned)((ckv_scan_blocks(P, n) + P.scan_tile - 1) >> P.lg_tile);
    tot += t;
    if (i < s) before += t;
    if (i == s) { mine = t; n_mine = (unsigned)n; }
  }
  tot = __reduce_add_sync(0xffffffffu, tot);
  before = __reduce_add_sync(0xffffffffu, before);
  mine = __reduce_add_sync(0xffffffffu, mine);
  n_mine = __reduce_add_sync(0xffffffffu, n_mine);
  const unsigned T = tot * (unsigned)P.Hkv, T0 = before * (unsigned)P.Hkv + (unsigned)h * mine;
  const unsigned tpc = max(ckv_udiv24(T + (unsigned)scan_grid - 1u, (unsigned)scan_grid), 1u);
  const int cfirst = (int)ckv_udiv24(T0, tpc);
  const int ccount = mine == 0 ? 0 : (int)ckv_udiv24(T0 + mine - 1u, tpc) - cfirst + 1;
  first = (cfirst + 2 * unit) * CKV_SCAN_WARPS;
  count = ccount * CKV_SCAN_WARPS + ((P.tail && n_mine > 0) ? 1 : 0);
}
// The usual length source: the device array, clamped to the cache's capacity.
struct CkvClampedLens {
  const int *seq_lens;
  int cap;
  __device__ __forceinline__ int operator()(int i) const { return max(min(seq_lens[i], cap), 0); }
};

#endif  // __CUDACC__
