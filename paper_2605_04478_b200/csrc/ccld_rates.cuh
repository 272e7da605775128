// Counter changes per op from raw probe samples (Sec. 4.1.2: SendRate / RecvRate are reciprocals of the number of
// changes of SendCount / RecvCount seen by a probe that samples at a fixed period; Sec. 5.2 step 2 does this on the
// host's diagnostic thread). For sm_100a, streaming and HBM-bound:
//
//   k_tick_sums     per tile of ticks: how many ticks changed SendCount / RecvCount against the previous tick of the
//                   same rank (a rank's first tick never counts)
//   k_tile_scan     exclusive prefix over the tile sums (one CTA)
//   k_tick_prefix   inclusive prefix of the change indicators per tick: low word send, high word recv
//   k_record_rates  per record: two searches in its rank's tick times (the first starts from an even-spacing guess,
//                   the second from the first), then a difference of prefixes
//
// No kernel waits on another CTA: the prefix is three plain launches.
#pragma once
#include "ccld_device.cuh"

namespace ccld {

constexpr int RT_THREADS = 256;
constexpr int RT_PER = 8;                          // consecutive ticks per thread
constexpr int RT_TILE = RT_THREADS * RT_PER;

struct TickArgs {
  u64 n_ticks; u32 n_ranks;
  const u64* tick_off;                             // [n_ranks + 1]
  const i64* tick_ns; const u32 *send, *recv;      // [n_ticks], a rank's ticks contiguous and in time order
  u64* prefix;                                     // [n_ticks]
  u64* tile_sum;                                   // [tiles]
};

// the rank whose ticks contain tick i: the last r with tick_off[r] <= i
__device__ __forceinline__ u32 tick_owner(const u64* __restrict__ off, u32 n_ranks, u64 i) {
  u32 lo = 0, hi = n_ranks - 1;
  while (lo < hi) { const u32 mid = (lo + hi + 1) >> 1; if (off[mid] <= i) lo = mid; else hi = mid - 1; }
  return lo;
}

// Change indicators of the thread's RT_PER consecutive ticks, packed (send | recv << 32); returns their sum.
__device__ __forceinline__ u64 tick_indicators(const TickArgs& A, u64 i0, u64 (&ind)[RT_PER]) {
  u64 sum = 0;
#pragma unroll
  for (int k = 0; k < RT_PER; ++k) ind[k] = 0;
  if (i0 >= A.n_ticks) return 0;
  u32 s[RT_PER], r[RT_PER];
  const bool full = i0 + RT_PER <= A.n_ticks;
  if (full && ((reinterpret_cast<uintptr_t>(A.send + i0) | reinterpret_cast<uintptr_t>(A.recv + i0)) & 15) == 0) {
#pragma unroll
    for (int q = 0; q < RT_PER / 4; ++q) {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(A.send + i0) + q), b = __ldg(reinterpret_cast<const uint4*>(A.recv + i0) + q);
      s[4 * q] = a.x; s[4 * q + 1] = a.y; s[4 * q + 2] = a.z; s[4 * q + 3] = a.w;
      r[4 * q] = b.x; r[4 * q + 1] = b.y; r[4 * q + 2] = b.z; r[4 * q + 3] = b.w;
    }
  } else {
#pragma unroll
    for (int k = 0; k < RT_PER; ++k) { const bool in = i0 + k < A.n_ticks; s[k] = in ? __ldg(A.send + i0 + k) : 0u; r[k] = in ? __ldg(A.recv + i0 + k) : 0u; }
  }
  u32 ps = i0 ? __ldg(A.send + i0 - 1) : 0u, pr = i0 ? __ldg(A.recv + i0 - 1) : 0u;
  // where the current rank's ticks end, and whether tick i0 opens a rank
  u32 rk = tick_owner(A.tick_off, A.n_ranks, i0);
  u64 seg_end = A.tick_off[rk + 1];
  bool first = A.tick_off[rk] == i0;
#pragma unroll
  for (int k = 0; k < RT_PER; ++k) {
    const u64 i = i0 + k;
    if (i < A.n_ticks) {
      if (i == seg_end) {                          // the next rank that has ticks starts here
        first = true;
        for (u32 step = 0; step <= A.n_ranks && A.tick_off[rk + 1] <= i; ++step) ++rk;
        seg_end = A.tick_off[rk + 1];
      }
      if (!first) ind[k] = (u64)(s[k] != ps ? 1u : 0u) | ((u64)(r[k] != pr ? 1u : 0u) << 32);
      first = false; ps = s[k]; pr = r[k];
      sum += ind[k];
    }
  }
  return sum;
}

// exclusive prefix of v over the CTA (all threads call); *total = the CTA's sum
__device__ __forceinline__ u64 cta_exclusive_scan(u64 v, u64* total, u64* s_warp /*[RT_THREADS / 32 + 1]*/) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u64 inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) { const u64 o = __shfl_up_sync(0xFFFFFFFFu, inc, d); if (lane >= (u32)d) inc += o; }
  if (lane == 31) s_warp[wid] = inc;
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 run = 0;
    for (int q = 0; q < RT_THREADS / 32; ++q) { const u64 x = s_warp[q]; s_warp[q] = run; run += x; }
    s_warp[RT_THREADS / 32] = run;
  }
  __syncthreads();
  const u64 r = s_warp[wid] + inc - v;
  *total = s_warp[RT_THREADS / 32];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(RT_THREADS) k_tick_sums(TickArgs A) {
  __shared__ u64 s_warp[RT_THREADS / 32 + 1];
  u64 ind[RT_PER];
  const u64 v = tick_indicators(A, (u64)blockIdx.x * RT_TILE + (u64)threadIdx.x * RT_PER, ind);
  u64 total;
  cta_exclusive_scan(v, &total, s_warp);
  if (threadIdx.x == 0) A.tile_sum[blockIdx.x] = total;
}

__global__ void __launch_bounds__(RT_THREADS) k_tile_scan(u64* __restrict__ tile_sum, u64 n_tiles) {
  __shared__ u64 s_warp[RT_THREADS / 32 + 1];
  u64 carry = 0;
  for (u64 base = 0; base < n_tiles; base += RT_TILE) {          // RT_PER consecutive sums per thread and round
    const u64 i0 = base + (u64)threadIdx.x * RT_PER;
    u64 v[RT_PER], sum = 0;
#pragma unroll
    for (int k = 0; k < RT_PER; ++k) { v[k] = i0 + k < n_tiles ? tile_sum[i0 + k] : 0; sum += v[k]; }
    u64 total;
    u64 run = carry + cta_exclusive_scan(sum, &total, s_warp);
#pragma unroll
    for (int k = 0; k < RT_PER; ++k) { if (i0 + k < n_tiles) tile_sum[i0 + k] = run; run += v[k]; }
    carry += total;
  }
}

__global__ void __launch_bounds__(RT_THREADS) k_tick_prefix(TickArgs A) {
  __shared__ u64 s_warp[RT_THREADS / 32 + 1];
  u64 ind[RT_PER];
  const u64 i0 = (u64)blockIdx.x * RT_TILE + (u64)threadIdx.x * RT_PER;
  const u64 v = tick_indicators(A, i0, ind);
  u64 total;
  u64 run = A.tile_sum[blockIdx.x] + cta_exclusive_scan(v, &total, s_warp);
#pragma unroll
  for (int k = 0; k < RT_PER; ++k) { run += ind[k]; ind[k] = run; }
  if (i0 + RT_PER <= A.n_ticks) {
    ulonglong2* dst = reinterpret_cast<ulonglong2*>(A.prefix + i0);          // i0 is a multiple of 8: 64-byte aligned
#pragma unroll
    for (int q = 0; q < RT_PER / 2; ++q) dst[q] = make_ulonglong2(ind[2 * q], ind[2 * q + 1]);
  } else {
#pragma unroll
    for (int k = 0; k < RT_PER; ++k) if (i0 + k < A.n_ticks) A.prefix[i0 + k] = ind[k];
  }
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
  u64 g = (u64)((double)(t - t0) / (double)(t1 - t0) * (double)(n - 1));
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
      const u64 ca = ticks_upto_guess(A.tick_ns, lo, hi, a);
      const u64 cb = b == -1 ? hi - lo : (b < a ? 0 : ca + ticks_upto_near(A.tick_ns, lo + ca, hi, b));
      // a rank's first tick has no indicator, so the prefix "before the first tick" equals the prefix at it
      const u64 ia = lo + (ca ? ca - 1 : 0), ib = lo + (cb ? cb - 1 : 0);
      if (ib > ia) {
        const u64 pa = A.prefix[ia], pb = A.prefix[ib];
        s = (u32)pb - (u32)pa; q = (u32)(pb >> 32) - (u32)(pa >> 32);
      }
    }
  }
  send_chg[i] = s; recv_chg[i] = q;
}

}  // namespace ccld
