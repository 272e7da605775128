// Counter changes per op from raw probe samples (Sec. 4.1.2: SendRate / RecvRate are reciprocals of the number of
// changes of SendCount / RecvCount seen by a probe that samples at a fixed period; Sec. 5.2 step 2 does this on the
// host's diagnostic thread). For sm_100a, streaming and HBM-bound. The prefix of the change indicators is kept per
// block of 32 ticks - the count before the block plus one bit per tick - so the counters are read once and what is
// written is half a byte per tick:
//
//   k_tick_blocks   per block of 32 ticks: which ticks changed SendCount / RecvCount against the previous tick of the
//                   same rank (a rank's first tick never counts), as two 32-bit masks with their bit counts; per tile
//                   of 64 blocks the sum of the counts
//   k_tile_scan     exclusive prefix over the tile sums (one CTA)
//   k_block_prefix  exclusive prefix of the counts inside each tile plus the tile's offset
//   k_record_rates  per record: two searches in its rank's tick times (the first starts from an even-spacing guess,
//                   the second from the first), then a difference of prefixes, each a block entry and a bit count
//
// No kernel waits on another CTA: the prefix is three plain launches.
#pragma once
#include "ccld_device.cuh"

namespace ccld {

constexpr int RT_THREADS = 256;
constexpr int RT_PER = 8;
constexpr int RT_TILE = RT_THREADS * RT_PER;       // ticks per CTA of k_tick_blocks: 8 warps x RB_PER_WARP blocks x 32
constexpr int RB_PER_WARP = 8;
constexpr int RB_PER_TILE = RT_TILE / 32;          // 64 blocks

// x: changes before the block (send in the low word, recv in the high word; while k_tick_blocks runs: inside the block);
// y: change bits of the block's ticks (send low, recv high)
typedef ulonglong2 TickBlock;

struct TickArgs {
  u64 n_ticks; u32 n_ranks;
  const u64* tick_off;                             // [n_ranks + 1]
  const i64* tick_ns; const u32 *send, *recv;      // [n_ticks], a rank's ticks contiguous and in time order
  TickBlock* blk;                                  // [ceil(n_ticks / 32)]
  u64* tile_sum;                                   // [tiles]
};

// the rank whose ticks contain tick i: the last r with tick_off[r] <= i
__device__ __forceinline__ u32 tick_owner(const u64* __restrict__ off, u32 n_ranks, u64 i, u64 n_ticks) {
  // probes sample at one period, so the ranks' segments are about equally long: the proportional guess comes first
  const u32 g = (u32)min((u64)(n_ranks - 1), (u64)((double)i * (double)n_ranks / (double)n_ticks));
  const u64 g0 = off[g], g1 = off[g + 1];
  if (g0 <= i && i < g1) return g;
  u32 lo = 0, hi = n_ranks - 1;
  if (g0 <= i) lo = g; else hi = g ? g - 1 : 0;
  while (lo < hi) { const u32 mid = (lo + hi + 1) >> 1; if (off[mid] <= i) lo = mid; else hi = mid - 1; }
  return lo;
}

// One warp per RB_PER_WARP consecutive blocks, one lane per tick: the predecessor's counters come from the lane below
// (from the previous block's last lane, or from memory, for lane 0). Where the ranks' segments start is found once per
// warp (a proportional guess, else a search in the offset table) and then followed from block to block.
__global__ void __launch_bounds__(RT_THREADS) k_tick_blocks(TickArgs A) {
  __shared__ u64 s_cnt[RT_THREADS / 32];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const u64 t0 = (u64)blockIdx.x * RT_TILE + (u64)wid * (RB_PER_WARP * 32);
  u64 wsum = 0;
  if (t0 < A.n_ticks) {
    u32 rk = tick_owner(A.tick_off, A.n_ranks, t0, A.n_ticks);             // a rank that has ticks: t0 < n_ticks
    u64 seg_start = A.tick_off[rk], seg_end = A.tick_off[rk + 1];
    u32 carry_s = t0 ? __ldg(A.send + t0 - 1) : 0u, carry_r = t0 ? __ldg(A.recv + t0 - 1) : 0u;
    u32 sv_[RB_PER_WARP], rv_[RB_PER_WARP];                     // all loads of the warp's blocks are issued before the first is used
    if (t0 + RB_PER_WARP * 32 <= A.n_ticks && seg_start < t0 && seg_end >= t0 + RB_PER_WARP * 32) {
      // the usual case: all of the warp's ticks exist and lie inside one rank's segment, after its first tick
      const u32 *ps_ = A.send + t0 + lane, *pr_ = A.recv + t0 + lane;
#pragma unroll
      for (int q = 0; q < RB_PER_WARP; ++q) { sv_[q] = __ldg(ps_ + q * 32); rv_[q] = __ldg(pr_ + q * 32); }
      TickBlock* out = A.blk + (t0 >> 5);
#pragma unroll
      for (int q = 0; q < RB_PER_WARP; ++q) {
        u32 ps = __shfl_up_sync(0xFFFFFFFFu, sv_[q], 1), pr = __shfl_up_sync(0xFFFFFFFFu, rv_[q], 1);
        if (lane == 0) { ps = carry_s; pr = carry_r; }
        carry_s = __shfl_sync(0xFFFFFFFFu, sv_[q], 31); carry_r = __shfl_sync(0xFFFFFFFFu, rv_[q], 31);
        const u32 ms = __ballot_sync(0xFFFFFFFFu, sv_[q] != ps), mr = __ballot_sync(0xFFFFFFFFu, rv_[q] != pr);
        const u64 cnt = (u64)__popc(ms) | ((u64)__popc(mr) << 32);
        if (lane == 0) out[q] = make_ulonglong2(cnt, (u64)ms | ((u64)mr << 32));
        wsum += cnt;
      }
    } else {
#pragma unroll
    for (int q = 0; q < RB_PER_WARP; ++q) {
      const u64 i = t0 + (u64)q * 32 + lane;
      const bool in = i < A.n_ticks;
      sv_[q] = in ? __ldg(A.send + i) : 0u; rv_[q] = in ? __ldg(A.recv + i) : 0u;
    }
#pragma unroll
    for (int q = 0; q < RB_PER_WARP; ++q) {
      const u64 bstart = t0 + (u64)q * 32;
      if (bstart >= A.n_ticks) break;                           // the same in every lane
      const u64 bend = bstart + 32 < A.n_ticks ? bstart + 32 : A.n_ticks;
      const u64 i = bstart + lane;
      const bool in = i < A.n_ticks;
      const u32 sv = sv_[q], rv = rv_[q];
      u32 ps = __shfl_up_sync(0xFFFFFFFFu, sv, 1), pr = __shfl_up_sync(0xFFFFFFFFu, rv, 1);
      if (lane == 0) { ps = carry_s; pr = carry_r; }
      carry_s = __shfl_sync(0xFFFFFFFFu, sv, 31); carry_r = __shfl_sync(0xFFFFFFFFu, rv, 31);
      // first ticks of ranks inside [bstart, bend): the current segment's, if it starts here, and those of the segments
      // that start before the block ends (a rank without ticks has an empty segment and no first tick)
      bool first = seg_start >= bstart && i == seg_start;
      for (u32 step = 0; step <= A.n_ranks && seg_end < bend; ++step) {
        ++rk; seg_start = seg_end; seg_end = A.tick_off[rk + 1];
        if (seg_end > seg_start) first = first || i == seg_start;
      }
      const u32 ms = __ballot_sync(0xFFFFFFFFu, in && !first && sv != ps), mr = __ballot_sync(0xFFFFFFFFu, in && !first && rv != pr);
      const u64 cnt = (u64)__popc(ms) | ((u64)__popc(mr) << 32);
      if (lane == 0) A.blk[bstart >> 5] = make_ulonglong2(cnt, (u64)ms | ((u64)mr << 32));
      wsum += cnt;
    }
    }
  }
  if (lane == 0) s_cnt[wid] = wsum;
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 t = 0;
    for (int q = 0; q < RT_THREADS / 32; ++q) t += s_cnt[q];
    A.tile_sum[blockIdx.x] = t;
  }
}

// One CTA of 1,024 threads; a round covers 16,384 tiles (33.5 M ticks). A warp owns 512 consecutive sums of the round and
// reads them 32 at a time, lanes on consecutive sums (coalesced, all sixteen loads issued before the first is used), scans
// each 32 with shuffles and carries its running total from step to step; the warps' totals are scanned by every warp.
constexpr int TS_THREADS = 1024;
constexpr int TS_PER = 16;
__global__ void __launch_bounds__(TS_THREADS) k_tile_scan(u64* __restrict__ tile_sum, u64 n_tiles) {
  __shared__ u64 s_warp[TS_THREADS / 32];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u64 carry = 0;
  for (u64 base = 0; base < n_tiles; base += (u64)TS_THREADS * TS_PER) {
    const u64 i0 = base + (u64)wid * (32 * TS_PER) + lane;
    u64 v[TS_PER];
#pragma unroll
    for (int k = 0; k < TS_PER; ++k) v[k] = i0 + 32 * k < n_tiles ? tile_sum[i0 + 32 * k] : 0;
    u64 run = 0;                                      // the warp's sums before step k
#pragma unroll
    for (int k = 0; k < TS_PER; ++k) {
      u64 inc = v[k];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) { const u64 o = __shfl_up_sync(0xFFFFFFFFu, inc, d); if (lane >= (u32)d) inc += o; }
      v[k] = run + inc - v[k];                        // exclusive inside the warp's span
      run += __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    if (lane == 0) s_warp[wid] = run;
    __syncthreads();
    u64 w = s_warp[lane], winc = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const u64 o = __shfl_up_sync(0xFFFFFFFFu, winc, d); if (lane >= (u32)d) winc += o; }
    const u64 before = carry + __shfl_sync(0xFFFFFFFFu, winc - w, wid);
    carry += __shfl_sync(0xFFFFFFFFu, winc, 31);
#pragma unroll
    for (int k = 0; k < TS_PER; ++k) if (i0 + 32 * k < n_tiles) tile_sum[i0 + 32 * k] = before + v[k];
    __syncthreads();                                  // s_warp is written again in the next round
  }
}

// 64 threads: the counts of a tile's blocks become the changes before each block
__global__ void __launch_bounds__(RB_PER_TILE) k_block_prefix(TickArgs A) {
  __shared__ u64 s_half;
  const u64 n_blocks = (A.n_ticks + 31) >> 5;
  const u64 b = (u64)blockIdx.x * RB_PER_TILE + threadIdx.x;
  const u32 lane = threadIdx.x & 31;
  const u64 v = b < n_blocks ? A.blk[b].x : 0;
  u64 inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) { const u64 o = __shfl_up_sync(0xFFFFFFFFu, inc, d); if (lane >= (u32)d) inc += o; }
  if (threadIdx.x == 31) s_half = inc;
  __syncthreads();
  const u64 ex = A.tile_sum[blockIdx.x] + (threadIdx.x >= 32 ? s_half : 0) + inc - v;
  if (b < n_blocks) A.blk[b].x = ex;
}

// changes up to and including tick i (send in the low word, recv in the high word)
__device__ __forceinline__ u64 changes_upto(const TickBlock* __restrict__ blk, u64 i) {
  const TickBlock e = blk[i >> 5];
  const u32 keep = 0xFFFFFFFFu >> (31 - (u32)(i & 31));
  return e.x + (u64)__popc((u32)e.y & keep) + ((u64)__popc((u32)(e.y >> 32) & keep) << 32);
}

// ticks of [lo, hi) at or before t
__device__ __forceinline__ u64 ticks_upto(const i64* __restrict__ tn, u64 lo, u64 hi, i64 t) {
  u64 a = lo, b = hi;                              // first index in [lo, hi) with tn > t
  for (int step = 0; step < 64 && a < b; ++step) { const u64 mid = a + ((b - a) >> 1); if (__ldg(tn + mid) <= t) a = mid + 1; else b = mid; }
  return a - lo;
}

// the same count when it is expected to be small (an op spans a few ticks): doubling steps from lo, then bisection
__device__ __forceinline__ u64 ticks_upto_near(const i64* __restrict__ tn, u64 lo, u64 hi, i64 t) {
  u64 pos = lo, bound = 1;                          // every tick of [lo, pos) is at or before t
  for (int step = 0; step < 64 && pos + bound - 1 < hi && __ldg(tn + pos + bound - 1) <= t; ++step) { pos += bound; bound <<= 1; }
  const u64 end = pos + bound - 1 < hi ? pos + bound - 1 : hi;
  return (pos - lo) + ticks_upto(tn, pos, end, t);
}

// The same count, started from where t would sit if the ticks were evenly spaced (probes sample at a fixed period, so
// the guess is usually within a tick or two); doubling steps up or down from the guess, then bisection. Any spacing
// gives the right count: the guess only decides where the search starts.
__device__ __forceinline__ u64 ticks_upto_guess(const i64* __restrict__ tn, u64 lo, u64 hi, i64 t) {
  const u64 n = hi - lo;
  if (n == 0) return 0;
  const i64 t0 = __ldg(tn + lo), t1 = __ldg(tn + hi - 1);
  if (t < t0) return 0;
  if (t >= t1) return n;
  // tn[lo] <= t < tn[hi - 1]: the first tick after t has index j in [1, n - 1]
  u64 g = (u64)(__fdividef((float)(t - t0), (float)(t1 - t0)) * (float)(n - 1));   // single precision is plenty for a starting point
  g = g > n - 2 ? n - 2 : g;
  u64 j;
  if (__ldg(tn + lo + g) <= t) {
    u64 pos = g, step = 1;                          // tn[lo + pos] <= t
    for (int it = 0; it < 64 && pos + step < n && __ldg(tn + lo + pos + step) <= t; ++it) { pos += step; step <<= 1; }
    const u64 end = pos + step < n - 1 ? pos + step : n - 1;          // tn[lo + end] > t
    j = pos + 1 + ticks_upto(tn, lo + pos + 1, lo + end, t);
  } else {
    u64 pos = g, step = 1;                          // tn[lo + pos] > t
    for (int it = 0; it < 64 && pos >= step && __ldg(tn + lo + pos - step) > t; ++it) { pos -= step; step <<= 1; }
    const u64 start = pos >= step ? pos - step : 0;                   // tn[lo + start] <= t
    j = start + 1 + ticks_upto(tn, lo + start + 1, lo + pos, t);
  }
  return j;
}

// The same three searches with 32-bit indices relative to the start of a rank's segment (segments of fewer than 2^32
// ticks, which is every segment that fits a GPU's memory next to its records; longer ones take the 64-bit forms above).
__device__ __forceinline__ u32 seg_upto(const i64* __restrict__ tn, u32 a, u32 b, i64 t) {      // first index of [a, b) whose tick is after t
  for (int step = 0; step < 32 && a < b; ++step) { const u32 mid = a + ((b - a) >> 1); if (__ldg(tn + mid) <= t) a = mid + 1; else b = mid; }
  return a;
}
__device__ __forceinline__ u32 seg_upto_near(const i64* __restrict__ tn, u32 from, u32 n, i64 t) {   // every tick of [0, from) is at or before t
  u32 pos = from, bound = 1;
  for (int step = 0; step < 32 && pos + bound - 1 < n && __ldg(tn + pos + bound - 1) <= t; ++step) { pos += bound; bound <<= 1; }
  const u32 end = pos + bound - 1 < n ? pos + bound - 1 : n;
  return seg_upto(tn, pos, end, t);
}
__device__ __forceinline__ u32 seg_upto_guess(const i64* __restrict__ tn, u32 n, i64 t) {
  const i64 t0 = __ldg(tn), t1 = __ldg(tn + n - 1);
  if (t < t0) return 0;
  if (t >= t1) return n;
  // tn[0] <= t < tn[n - 1]: the first tick after t has index j in [1, n - 1]
  u32 g = (u32)(__fdividef((float)(t - t0), (float)(t1 - t0)) * (float)(n - 1));
  g = g > n - 2 ? n - 2 : g;
  if (__ldg(tn + g) <= t) {
    u32 pos = g, step = 1;                          // tn[pos] <= t
    for (int it = 0; it < 32 && pos + step < n && __ldg(tn + pos + step) <= t; ++it) { pos += step; step <<= 1; }
    const u32 end = pos + step < n - 1 ? pos + step : n - 1;          // tn[end] > t
    return seg_upto(tn, pos + 1, end, t);
  }
  u32 pos = g, step = 1;                            // tn[pos] > t
  for (int it = 0; it < 32 && pos >= step && __ldg(tn + pos - step) > t; ++it) { pos -= step; step <<= 1; }
  const u32 start = pos >= step ? pos - step : 0;                     // tn[start] <= t
  return seg_upto(tn, start + 1, pos, t);
}

__global__ void __launch_bounds__(RT_THREADS) k_record_rates(TickArgs A, u64 n_rec, const u32* __restrict__ rank, const i64* __restrict__ t_enter,
                                                           const i64* __restrict__ t_exit, u32* __restrict__ send_chg, u32* __restrict__ recv_chg) {
  const u64 i = (u64)blockIdx.x * RT_THREADS + threadIdx.x;
  if (i >= n_rec) return;
  const u32 r = rank[i];
  u32 s = 0, q = 0;
  if (r < A.n_ranks) {
    const u64 lo = A.tick_off[r], hi = A.tick_off[r + 1];
    if (hi > lo) {
      const i64 a = t_enter[i], b = t_exit[i];
      u64 ca, cb;
      if (hi - lo < 0xFFFFFFFFull) {
        const i64* __restrict__ tn = A.tick_ns + lo; const u32 n = (u32)(hi - lo);
        const u32 xa = seg_upto_guess(tn, n, a);
        ca = xa; cb = b == -1 ? n : (b < a ? 0u : seg_upto_near(tn, xa, n, b));
      } else {
        ca = ticks_upto_guess(A.tick_ns, lo, hi, a);
        cb = b == -1 ? hi - lo : (b < a ? 0 : ca + ticks_upto_near(A.tick_ns, lo + ca, hi, b));
      }
      // a rank's first tick has no indicator, so the prefix "before the first tick" equals the prefix at it
      const u64 ia = lo + (ca ? ca - 1 : 0), ib = lo + (cb ? cb - 1 : 0);
      if (ib > ia) {
        const u64 pa = changes_upto(A.blk, ia), pb = changes_upto(A.blk, ib);
        s = (u32)pb - (u32)pa; q = (u32)(pb >> 32) - (u32)(pa >> 32);
      }
    }
  }
  send_chg[i] = s; recv_chg[i] = q;
}

}  // namespace ccld
