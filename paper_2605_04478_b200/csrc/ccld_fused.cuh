// Per-op reductions, median / MAD, flags and votes for communicators of up to 128 ranks (sm_100a).
//
//   k_reduce_fused     the common case: every member reported, nothing in flight, all times of the group within
//                      2^31 ns of its first member's enter time. A group sits in L = n_pad / 8 lanes of a warp, eight
//                      ring positions per lane (n <= 8: one thread per group, lanes along consecutive op counters so
//                      that the gathers of one member coalesce). Times become 32-bit offsets as they arrive and are
//                      parked in shared memory, so that a thread never holds more than one batch of gathers plus
//                      one set of eight sort keys in registers: three CTAs of 256 threads fit an SM. Any other
//                      group is appended to a list.
//   k_reduce_deferred  the listed groups, one warp each, in full 64-bit generality: missing members, records in
//                      flight (hang alerts), invalid times, spreads beyond 32 bits.
//
// The work list of k_reduce_fused is chunk-major (see k_plan), so CTAs that run together gather from the same stretch
// of every rank's records and share the fetched sectors in L2.
#pragma once
#include "ccld_device.cuh"

namespace ccld {

constexpr u32 FULLM = 0xFFFFFFFFu;
#ifndef CCLD_FUSED_MIN_CTAS
#define CCLD_FUSED_MIN_CTAS 3
#endif

template <class K> __device__ __forceinline__ void cswap(K& a, K& b) { const K lo = min(a, b), hi = max(a, b); a = lo; b = hi; }
__device__ __forceinline__ u32 key_absdiff(u32 a, u32 b) { return __usad(a, b, 0u); }
__device__ __forceinline__ u64 key_absdiff(u64 a, u64 b) { return a >= b ? a - b : b - a; }

// 19-exchange sorting network for 8 keys
template <class K> __device__ __forceinline__ void sort8(K (&v)[8]) {
  cswap(v[0], v[2]); cswap(v[1], v[3]); cswap(v[4], v[6]); cswap(v[5], v[7]);
  cswap(v[0], v[4]); cswap(v[1], v[5]); cswap(v[2], v[6]); cswap(v[3], v[7]);
  cswap(v[0], v[1]); cswap(v[2], v[3]); cswap(v[4], v[5]); cswap(v[6], v[7]);
  cswap(v[2], v[4]); cswap(v[3], v[5]);
  cswap(v[1], v[4]); cswap(v[3], v[6]);
  cswap(v[1], v[2]); cswap(v[3], v[4]); cswap(v[5], v[6]);
}
// bitonic merge: sorts 8 keys that first fall and then rise
template <class K> __device__ __forceinline__ void merge8(K (&v)[8]) {
  cswap(v[0], v[4]); cswap(v[1], v[5]); cswap(v[2], v[6]); cswap(v[3], v[7]);
  cswap(v[0], v[2]); cswap(v[1], v[3]); cswap(v[4], v[6]); cswap(v[5], v[7]);
  cswap(v[0], v[1]); cswap(v[2], v[3]); cswap(v[4], v[5]); cswap(v[6], v[7]);
}
template <class K> __device__ __forceinline__ K pick4(const K (&v)[8], u32 k) {
  K r = v[0];
  r = k == 1 ? v[1] : r; r = k == 2 ? v[2] : r; r = k == 3 ? v[3] : r;
  return r;
}

template <class K> struct KeyMax;
template <> struct KeyMax<u32> { static __device__ __forceinline__ u32 v() { return 0xFFFFFFFFu; } };
template <> struct KeyMax<u64> { static __device__ __forceinline__ u64 v() { return U64_MAX_; } };

// lower median and lower-median absolute deviation of x[0..n), n <= 8 (x[p] = maximum key for p >= n)
template <class K> __device__ __forceinline__ void median_mad8(const K (&x)[8], u32 n, K* med, K* mad) {
  K s[8];
#pragma unroll
  for (int p = 0; p < 8; ++p) s[p] = x[p];
  sort8(s);
  const u32 k = (n - 1) >> 1;
  const K m = pick4(s, k);
#pragma unroll
  for (int p = 0; p < 8; ++p) s[p] = (u32)p < n ? key_absdiff(s[p], m) : KeyMax<K>::v();   // falls to 0 at k, then rises
  merge8(s);
  *med = m; *mad = pick4(s, k);
}

// 1 / x for x >= 1 to within a few ulp: single-precision seed and two Newton steps
// one Newton step on the single-precision seed: relative error near 2e-14
__device__ __forceinline__ float rcp_seed(double x) {     // 1 <= x < 2^64: the approximate reciprocal is good to about 2^-22
  float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"((float)x)); return r;
}
__device__ __forceinline__ double rcp_newton1(double x) {
  const double r = (double)rcp_seed(x);
  return fma(r, fma(-x, r, 1.0), r);
}
__device__ __forceinline__ double rcp_newton(double x) {
  double r = (double)rcp_seed(x);
  double e = fma(-x, r, 1.0); r = fma(r, e, r);
  e = fma(-x, r, 1.0); r = fma(r, e, r);
  return r;
}
__device__ __forceinline__ double busbw_fast(double bytes_num, double den, i64 t) {
  return t > 0 ? bytes_num * rcp_newton((double)t * den) : 0.0;
}

// Sums v[m] over the warp for m = 0..7 with 9 shuffles; lane l ends up with the total of member
// m = 4 * bit4(l) + 2 * bit3(l) + bit2(l).
__device__ __forceinline__ double warp_sum8(double (&v)[8], u32 lane) {
#pragma unroll
  for (int w = 4, bit = 16; w >= 1; w >>= 1, bit >>= 1) {
    const bool hi = (lane & bit) != 0;
#pragma unroll
    for (int i = 0; i < w; ++i) {
      const double send = hi ? v[i] : v[i + w], keep = hi ? v[i + w] : v[i];
      v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, bit);
    }
  }
  v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 2);
  v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
  return v[0];
}

template <class K> __device__ __forceinline__ K pick8(const K (&v)[8], u32 r) {
  K x = v[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) x = r == (u32)i ? v[i] : x;
  return x;
}

// One cross-lane step of a merge network: element r of this lane against element r (MIRROR: 7 - r) of lane ^ mask;
// the lane with keep_low set keeps the smaller key of each pair.
template <class K, bool MIRROR>
__device__ __forceinline__ void sub_exchange(K (&v)[8], int mask, bool keep_low) {
  K o[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) o[r] = __shfl_xor_sync(0xFFFFFFFFu, v[MIRROR ? 7 - r : r], mask);
#pragma unroll
  for (int r = 0; r < 8; ++r) v[r] = keep_low ? min(v[r], o[r]) : max(v[r], o[r]);
}

// Sorts the 8 L keys of a group ascending; element i lives in lane i / 8 (of the group), register i % 8.
template <int L, class K>
__device__ __forceinline__ void sub_sort(K (&v)[8], u32 s) {
  sort8(v);
#pragma unroll
  for (int m = 1; m < L; m <<= 1) {
    // two ascending runs of m lanes each: the mirror step leaves every key of the low run <= every key of the high
    // run and both runs bitonic; half-cleaners across lanes and then inside the lane finish the merge
    sub_exchange<K, true>(v, 2 * m - 1, (s & m) == 0);
#pragma unroll
    for (int h = m >> 1; h >= 1; h >>= 1) sub_exchange<K, false>(v, h, (s & h) == 0);
    merge8(v);
  }
}
// Sorts 8 L keys that fall and then rise.
template <int L, class K>
__device__ __forceinline__ void sub_merge(K (&v)[8], u32 s) {
#pragma unroll
  for (int h = L >> 1; h >= 1; h >>= 1) sub_exchange<K, false>(v, h, (s & h) == 0);
  merge8(v);
}

// Lower median and lower-median absolute deviation of a group's keys (x[q] = maximum key where the position does
// not exist or the group is not sorted at all). Every lane of the warp must call it.
template <int L, class K>
__device__ __forceinline__ void sub_median_mad(const K (&x)[8], u32 n, u32 s, u32 lane, K* med, K* mad) {
  K v[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) v[q] = x[q];
  sub_sort<L, K>(v, s);
  const u32 k = (n - 1) >> 1, src = (lane & ~(u32)(L - 1)) | (k >> 3);
  const K m = __shfl_sync(0xFFFFFFFFu, pick8(v, k & 7), src);
#pragma unroll
  for (int r = 0; r < 8; ++r) v[r] = s * 8 + r < n ? key_absdiff(v[r], m) : KeyMax<K>::v();   // falls to 0 at k, then rises
  sub_merge<L, K>(v, s);
  *med = m; *mad = __shfl_sync(0xFFFFFFFFu, pick8(v, k & 7), src);
}


// Per-lane running totals of the groups a warp has handled. Group counts live in the first lane of each group, six
// bits each; flag counts in the lane of the record, sixteen bits each.
struct FastAcc {
  u32 groups = 0;          // complete | barrier << 6 | analysed << 12 | mismatch << 18 | round << 24
  u32 flagged = 0;         // skew flags | duration flags << 16
  u32 n_def = 0;
  u32 best_rng = 0, best_k = NONE;
};
enum { FA_COMP = 0, FA_BAR = 6, FA_AN = 12, FA_MIS = 18, FA_ROUND = 24 };
enum { SC_COMP = 0, SC_INC, SC_BAR, SC_AN, SC_MIS, SC_PRES, SC_FS, SC_FD, SC_COUNT };

struct DeferList { u64* entries; u32* count; };    // entry: window index in the batch << 32 | group index in the window

// Where a window's outputs go; kept in shared memory and read when a group stores, so that the pointers do not occupy
// registers across the gathers.
struct OutPtrs { u8* flags; i64* gi64; u32* gu32; double* gbw; u64 G; };
template <class T> __device__ __forceinline__ T ld_volatile(const T& x) { return *(const volatile T*)&x; }

struct FusedShared {
  double bw[SMALL_SEQS / 32][WARP_N];
  u32 comm[SMALL_SEQS / 32], rounds[SMALL_SEQS / 32], n_an[SMALL_SEQS / 32], n_def[SMALL_SEQS / 32], brng[SMALL_SEQS / 32], bk[SMALL_SEQS / 32];
  u32 cnt[SC_COUNT];
  OutPtrs out;
  // n <= 32: per thread (column) eight enter-time offsets and eight durations. 33 <= n <= 128: the tile's keys as
  // [metric][member][op counter], pitch S + 1 (S = op counters per tile), written by the staging phase of the tile.
  u32 stage[2 * (MID_ELEMS + WARP_N)];
  u64 t_base[32], t_gby[32], t_ck[SMALL_SEQS / 32][32];       // staged tiles, per op counter: time base, size of the op, most changes per warp
  u32 t_gop[32], t_bits[32];                                  //   op code; 1 = some record disqualifies the group, 2 = the op set differs
};
constexpr u32 STAGE_ROWS = SMALL_SEQS;                        // row pitch of the per-thread layout

// Staging phase of a tile of a communicator of 33 to 128 ranks (S = 2048 / n_pad op counters, S <= 32): the CTA's warps
// share the members, lanes run along the op counter, so the record indices of a warp step are one contiguous piece of
// the member-major permutation and - in a rank-major upload - the records themselves lie in one short stretch of a
// rank's stream instead of one sector per lane. Times become 32-bit keys against the group's first member (whose enter
// time, size and op code every thread loads for its own op counter), the op-set check and the rate column are reduced on
// the way; the keys land in shared memory as [metric][member][op counter].
template <int L>
__device__ __forceinline__ void stage_tile(const WinDesc& D, const RangeRow& row, u32 seq0, u32 count, FusedShared& sh) {
  constexpr u32 S = 32 / L * (SMALL_SEQS / 32), PITCH = S + 1, NW = SMALL_SEQS / 32;     // S op counters per tile: 32 (n_pad 64), 16 (n_pad 128)
  constexpr u32 MPS = 32 / S;                                  // members a warp step covers
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5, n = row.n;
  const u32 sq = lane & (S - 1), ml = lane / S;
  const bool sv = sq < count;
  const u32* __restrict__ perm = D.perm + row.slot0 + seq0 + (sv ? sq : 0u);
  const i64* __restrict__ c_te = D.t_enter; const i64* __restrict__ c_tx = D.t_exit;
  const u64* __restrict__ c_by = D.bytes; const u8* __restrict__ c_op = D.op;
  const u32* __restrict__ c_sc = D.send_chg; const u32* __restrict__ c_rc = D.recv_chg;
  u32 bits = 0; i64 te0 = 0; u64 by0 = 0; u32 op0 = 0;
  {
    const u32 i0 = sv ? __ldg(perm) : NONE;
    if (i0 != NONE) { te0 = c_te[i0]; by0 = c_by[i0]; op0 = c_op[i0]; } else bits = 1;
  }
  const u64 base = (u64)te0 - 0x80000000ull;
  u64 ck = 0;
  u32* __restrict__ k_a = sh.stage; u32* __restrict__ k_d = sh.stage + (MID_ELEMS + WARP_N);
  // member of warp step i: wid * MPS + ml + i * NW * MPS
  for (u32 p0 = wid * MPS + ml; p0 < n; p0 += 4 * NW * MPS) {
    u32 idx[4]; i64 x[4], y[4]; u64 by[4]; u32 op[4], ch[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) { const u32 p = p0 + q * NW * MPS; idx[q] = (sv && p < n) ? __ldg(perm + (u64)p * row.n_seq) : NONE; }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 ix = idx[q] == NONE ? 0u : idx[q];
      x[q] = c_te[ix]; y[q] = c_tx[ix]; by[q] = c_by[ix]; op[q] = c_op[ix]; ch[q] = 0;
      if (c_sc != nullptr) { const u32 sc = c_sc[ix], rc = c_rc[ix]; ch[q] = max(sc, rc); }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 p = p0 + q * NW * MPS;
      if (p < n) {
        u32 a_lo = 0, d = 0;
        if (idx[q] == NONE) { if (sv) bits |= 1; }
        else {
          const u64 ra = (u64)x[q] - base, rb = (u64)y[q] - base;
          a_lo = (u32)ra; const u32 b_lo = (u32)rb; d = b_lo - a_lo;
          if (((ra | rb) >> 32) != 0 || (x[q] | y[q]) < 0 || b_lo < a_lo) bits |= 1;     // beyond 32 bits, negative or in flight, exit before enter
          if (op[q] != op0 || by[q] != by0) bits |= 2;
          const u64 k2 = ((u64)ch[q] << 32) | (u64)(NONE - p); ck = k2 > ck ? k2 : ck;     // most changes, then the lowest position
        }
        k_a[p * PITCH + sq] = a_lo; k_d[p * PITCH + sq] = d;
      }
    }
  }
  if (MPS > 1) {                                              // the lanes that share an op counter
#pragma unroll
    for (u32 h = S; h < 32; h <<= 1) { bits |= __shfl_xor_sync(FULLM, bits, h); const u64 o = shfl_xor64(ck, h); ck = o > ck ? o : ck; }
  }
  if (lane < S) {
    sh.t_ck[wid][lane] = ck;
    if (bits) atomicOr(&sh.t_bits[lane], bits);
    if (wid == 0) { sh.t_base[lane] = base; sh.t_gby[lane] = by0; sh.t_gop[lane] = op0; }
  }
}

// One group per L lanes, eight ring positions per lane (position s * 8 + q in lane s of the group); the warp takes
// 32 / L consecutive op counters starting at offset seq0 of the communicator's range, `count` of them valid.
// FULL: the communicator fills every position (n = 8 L). STAGED: the tile's keys and per-op values wait in shared memory
// (stage_tile); jt0 = the warp's first op counter inside the tile.
template <int L, bool FULL, bool STAGED = false>
__device__ __forceinline__ void fast_groups(const WinDesc& D, u32 w_idx, const RangeRow& row, const u32* __restrict__ mem, u32 seq0, u32 count,
                                            const Registry& R, const Params& P, const DeferList& DL, FusedShared& sh, FastAcc& acc, double (&bw)[8],
                                            u32 jt0 = 0) {
  const u32 lane = threadIdx.x & 31, s = lane % L, j = lane / L, base_lane = lane - s, p0 = s * 8;
  const u32 gmask = L == 32 ? FULLM : (((1u << (L & 31)) - 1u) << base_lane);
  const u32 n = FULL ? (u32)(L * 8) : row.n;
  const bool active = j < count, lead = s == 0;
  constexpr u32 S_T = STAGED ? 32 / L * (SMALL_SEQS / 32) : 1, PITCH = S_T + 1;
  // where the keys of my eight positions are: a column of the per-thread layout, or rows of the staged tile
  const u32 jt = STAGED ? (active ? jt0 + j : jt0) : 0u;
  const u32* __restrict__ ka = STAGED ? sh.stage + p0 * PITCH + jt : &sh.stage[threadIdx.x];
  const u32* __restrict__ kd = STAGED ? sh.stage + (MID_ELEMS + WARP_N) + p0 * PITCH + jt : &sh.stage[8 * STAGE_ROWS + threadIdx.x];
  constexpr u32 KSTEP = STAGED ? PITCH : STAGE_ROWS;
  u32* __restrict__ my = &sh.stage[threadIdx.x];              // my[q * SMALL_SEQS]: offset of position q, my[(8 + q) * SMALL_SEQS]: duration

  bool ok = true;
  u32 emin = 0xFFFFFFFFu, emax = 0, xmax = 0, tmx = 0, tmn = 0xFFFFFFFFu;
  u64 base;
  bool mm = false;
  u64 gby, ck = 0; u32 gop;
  // thread per group: lane m fetches the rank of ring position m now, so that the ranks a row names are a shuffle away
  // when the row is written instead of one more round trip to memory
  u32 mem_l = 0;
  if (L == 1) mem_l = lane < n ? __ldg(mem + lane) : 0u;
  if (STAGED) {
    base = sh.t_base[jt]; gby = sh.t_gby[jt]; gop = sh.t_gop[jt];
    const u32 bits = sh.t_bits[jt];
    ok = !(bits & 1); mm = (bits & 2) != 0;
#pragma unroll
    for (int w = 0; w < SMALL_SEQS / 32; ++w) { const u64 o = sh.t_ck[w][jt]; ck = o > ck ? o : ck; }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (FULL || p0 + q < n) {
        const u32 a_lo = ka[q * KSTEP], d = kd[q * KSTEP];
        emin = min(emin, a_lo); emax = max(emax, a_lo); xmax = max(xmax, a_lo + d);
        tmx = max(tmx, d); tmn = min(tmn, d);
      }
    }
  } else {
  // ---- record indices of my eight positions (member-major permutation: stride n_seq) ----
  u32 idx[8];
  {
    const u32* __restrict__ pm = D.perm + row.slot0 + (u64)p0 * row.n_seq + seq0 + (active ? j : 0u);
#pragma unroll
    for (int q = 0; q < 8; ++q) idx[q] = (active && (FULL || p0 + q < n)) ? __ldg(pm + (u64)q * row.n_seq) : NONE;
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) if ((FULL || p0 + q < n) && idx[q] == NONE) ok = false;      // a missing member: the group is deferred

  // ---- batch 1: times, turned into 32-bit offsets from (first member's enter time - 2^31 ns) as they arrive ----
  {
    const i64* __restrict__ c_te = D.t_enter; const i64* __restrict__ c_tx = D.t_exit;
    i64 ta[8], tb[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) { const u32 ix = idx[q] == NONE ? 0u : idx[q]; ta[q] = c_te[ix]; tb[q] = c_tx[ix]; }
    base = (L == 1 ? (u64)ta[0] : __shfl_sync(FULLM, (u64)ta[0], base_lane)) - 0x80000000ull;
    u32 hx = 0, neg = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const u64 ra = (u64)ta[q] - base, rb = (u64)tb[q] - base;
      const u32 a_lo = (u32)ra, b_lo = (u32)rb, d = b_lo - a_lo;
      my[q * SMALL_SEQS] = a_lo; my[(8 + q) * SMALL_SEQS] = d;
      if (FULL || p0 + q < n) {
        hx |= (u32)(ra >> 32) | (u32)(rb >> 32);
        neg |= (u32)((u64)ta[q] >> 32) | (u32)((u64)tb[q] >> 32);
        if (b_lo < a_lo) ok = false;
        emin = min(emin, a_lo); emax = max(emax, a_lo); xmax = max(xmax, b_lo);
        tmx = max(tmx, d); tmn = min(tmn, d);
      }
    }
    if (hx != 0 || (int)neg < 0) ok = false;       // beyond 32 bits, negative, or in flight (t_exit = -1)
  }
  // ---- batch 2: op set (every member against the group's first) and rate column ----
  {
    const u64* __restrict__ c_by = D.bytes; const u8* __restrict__ c_op = D.op;
    const u32* __restrict__ c_sc = D.send_chg; const u32* __restrict__ c_rc = D.recv_chg;
    u64 by[8]; u32 op[8], ch[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const u32 ix = idx[q] == NONE ? 0u : idx[q];
      by[q] = c_by[ix]; op[q] = c_op[ix]; ch[q] = 0;
      if (c_sc != nullptr) { const u32 sc = c_sc[ix], rc = c_rc[ix]; ch[q] = max(sc, rc); }
    }
    gby = L == 1 ? by[0] : __shfl_sync(FULLM, by[0], base_lane);
    gop = L == 1 ? op[0] : __shfl_sync(FULLM, op[0], base_lane);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (FULL || p0 + q < n) {
        if (op[q] != gop || by[q] != gby) mm = true;
        const u64 k2 = ((u64)ch[q] << 32) | (u64)(NONE - (p0 + q));          // most changes, then the lowest position
        ck = k2 > ck ? k2 : ck;
      }
    }
  }
  }
  // ---- the lanes of a group meet ----
  bool gok = active && ok;
  if (L > 1) { const u32 b_ok = __ballot_sync(FULLM, ok); gok = active && (b_ok & gmask) == gmask; }     // every lane votes
  if (active && !gok && lead) {
    const u32 e = atomicAdd(DL.count, 1u);
    DL.entries[e] = ((u64)w_idx << 32) | (u64)(row.group0 + seq0 + j);
    ++acc.n_def;
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) bw[q] = 0.0;
  if (!__any_sync(FULLM, gok)) return;
  if (L > 1) {
#pragma unroll
    for (int h = 1; h < L; h <<= 1) {
      emin = min(emin, __shfl_xor_sync(FULLM, emin, h)); emax = max(emax, __shfl_xor_sync(FULLM, emax, h));
      xmax = max(xmax, __shfl_xor_sync(FULLM, xmax, h));
      tmx = max(tmx, __shfl_xor_sync(FULLM, tmx, h)); tmn = min(tmn, __shfl_xor_sync(FULLM, tmn, h));
      if (!STAGED) { const u64 o = shfl_xor64(ck, h); ck = o > ck ? o : ck; }
    }
  }
  // lowest position that holds the longest / shortest duration
  u32 pmax = NONE, pmin = NONE;
#pragma unroll
  for (int q = 7; q >= 0; --q) {
    if (FULL || p0 + q < n) { const u32 d = kd[q * KSTEP]; if (d == tmx) pmax = p0 + q; if (d == tmn) pmin = p0 + q; }
  }
  u32 r_tmin = 0, r_tmax = 0, r_chg = 0;                      // ranks the row names
  if (L == 1) {                                             // all lanes are still here
    r_tmin = __shfl_sync(FULLM, mem_l, pmin & 31u); r_tmax = __shfl_sync(FULLM, mem_l, pmax & 31u); r_chg = __shfl_sync(FULLM, mem_l, (NONE - (u32)ck) & 31u);
  }
  bool mismatch = mm;
  if (L > 1) {
#pragma unroll
    for (int h = 1; h < L; h <<= 1) { pmax = min(pmax, __shfl_xor_sync(FULLM, pmax, h)); pmin = min(pmin, __shfl_xor_sync(FULLM, pmin, h)); }
    if (!STAGED) mismatch = (__ballot_sync(FULLM, mm) & gmask) != 0;
  }
  const bool barrier = gop == CCLD_OP_ALLREDUCE && gby < P.barrier_bytes;
  const bool analysed = gok && !barrier && n >= P.min_group;

  // ---- order statistics: one metric at a time, keys read back from shared memory ----
  u32 ms = 0, ds = 0, md = 0, dm = 0;
  if (__any_sync(FULLM, analysed)) {
    u32 v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = (FULL || p0 + q < n) ? ka[q * KSTEP] - emin : 0xFFFFFFFFu;
    if (L == 1) median_mad8<u32>(v, n, &ms, &ds); else sub_median_mad<L, u32>(v, n, s, lane, &ms, &ds);
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = (FULL || p0 + q < n) ? kd[q * KSTEP] - tmn : 0xFFFFFFFFu;
    if (L == 1) median_mad8<u32>(v, n, &md, &dm); else sub_median_mad<L, u32>(v, n, s, lane, &md, &dm);
    if (!analysed) { ms = ds = md = dm = 0; }
  }
  if (!gok) return;

  // ---- flags, votes, per-member bandwidth ----
  double num, den; bus_factor(gop, n, &num, &den);
  const double bn = (double)gby * num;
  u32 f_lo = 0, f_hi = 0;                                   // my eight flag bytes
  {
    // |x - med| * 1000 > k * MAD, exact: deviations and MADs are below 2^32, so both sides fit 64 bits, and for whole
    // numbers a * 1000 > T is a > floor(T / 1000); a quotient of 2^32 - 1 or more can never be exceeded
    const u64 qs = (u64)ds * P.k_milli / 1000u, qd = (u64)dm * P.k_milli / 1000u;
    const u32 ts = qs > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)qs, td = qd > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)qd;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (FULL || p0 + q < n) {
        const u32 d = kd[q * KSTEP];
        const u32 sk = ka[q * KSTEP] - emin, dd = d - tmn;
        const u32 f = (__usad(sk, ms, 0u) > ts ? (u32)CCLD_F_SKEW_OUT : 0u) | (__usad(dd, md, 0u) > td ? (u32)CCLD_F_DUR_OUT : 0u) |
                      (sk > ms ? (u32)CCLD_F_SKEW_HI : 0u) | (dd > md ? (u32)CCLD_F_DUR_HI : 0u);
        if (q < 4) f_lo |= f << (8 * q); else f_hi |= f << (8 * (q - 4));
        if (!barrier && d != 0) bw[q] = bn * rcp_newton1((double)d * den);
      }
    }
    if (!analysed) {
      // every position that exists carries the not-analysed mark
      const u32 cnt = FULL ? 8u : (n > p0 ? (n - p0 < 8u ? n - p0 : 8u) : 0u);
      f_lo = 0x80808080u & (cnt >= 4 ? 0xFFFFFFFFu : (1u << (8 * cnt)) - 1u);
      f_hi = cnt > 4 ? 0x80808080u & (cnt >= 8 ? 0xFFFFFFFFu : (1u << (8 * (cnt - 4))) - 1u) : 0u;
    }
    // votes: outliers are rare, so they are taken off the flag bytes afterwards, one set bit at a time
    static_assert(CCLD_F_SKEW_OUT == 1 && CCLD_F_DUR_OUT == 2 && CCLD_F_SKEW_HI == 4 && CCLD_F_DUR_HI == 8, "flag bit layout");
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const u32 fw = half ? f_hi : f_lo;
      u32 o = fw & 0x03030303u;
      while (o) {
        const u32 b = (u32)__ffs(o) - 1u, q = (b >> 3) + 4u * half, dur = b & 1u;
        const u32 hi = (fw >> (b + 2u)) & 1u;               // the HI bit of the same metric sits two places up
        atomicAdd(&R.votes[(u64)mem[p0 + q] * 4 + 2u * dur + (hi ? 0u : 1u)], 1u);
        o &= o - 1u;
      }
    }
    acc.flagged += (u32)__popc(f_lo & 0x01010101u) + (u32)__popc(f_hi & 0x01010101u) +
                   (((u32)__popc(f_lo & 0x02020202u) + (u32)__popc(f_hi & 0x02020202u)) << 16);
  }
  {
    u8* __restrict__ fp = ld_volatile(sh.out.flags) + row.slot0 + (u64)(seq0 + j) * n + p0;
    if ((FULL || p0 + 8 <= n) && (reinterpret_cast<uintptr_t>(fp) & 7) == 0) *reinterpret_cast<uint2*>(fp) = make_uint2(f_lo, f_hi);
    else {
#pragma unroll
      for (int q = 0; q < 8; ++q) if (FULL || p0 + q < n) fp[q] = (u8)((q < 4 ? f_lo >> (8 * q) : f_hi >> (8 * (q - 4))) & 0xFFu);
    }
  }
  if (L > 1) { r_tmin = mem[pmin]; r_tmax = mem[pmax]; r_chg = mem[NONE - (u32)ck]; }
  if (lead) {
    const u64 g = row.group0 + seq0 + j, G = ld_volatile(sh.out.G);
    i64* __restrict__ gi = ld_volatile(sh.out.gi64) + g; u32* __restrict__ gu = ld_volatile(sh.out.gu32) + g;
    const u32 span = xmax - emin;
    gi[(u64)GI_E_MIN * G] = (i64)(base + emin); gi[(u64)GI_ARRIVAL_SKEW * G] = (i64)(u64)(emax - emin);
    gi[(u64)GI_T_MAX * G] = (i64)(u64)tmx; gi[(u64)GI_T_MIN * G] = (i64)(u64)tmn; gi[(u64)GI_SPAN * G] = (i64)(u64)span;
    gi[(u64)GI_MED_SKEW * G] = (i64)(u64)ms; gi[(u64)GI_MAD_SKEW * G] = (i64)(u64)ds;
    gi[(u64)GI_MED_DUR * G] = analysed ? (i64)((u64)tmn + md) : 0; gi[(u64)GI_MAD_DUR * G] = (i64)(u64)dm;
    gu[(u64)GU_RANK_TMIN * G] = r_tmin; gu[(u64)GU_RANK_TMAX * G] = r_tmax;
    gu[(u64)GU_MAX_CHG * G] = (u32)(ck >> 32); gu[(u64)GU_RANK_MAX_CHG * G] = r_chg;
    gu[(u64)GU_N_PRESENT * G] = n;
    gu[(u64)GU_GFLAGS * G] = CCLD_G_COMPLETE | (barrier ? CCLD_G_BARRIER : 0) | (mismatch ? CCLD_G_OPSET_MISMATCH : 0) | (analysed ? CCLD_G_ANALYSED : 0);
    ld_volatile(sh.out.gbw)[g] = span ? bn * rcp_newton((double)span * den) : 0.0;
    acc.groups += (1u << FA_COMP) | (barrier ? 1u << FA_BAR : 0u) | (analysed ? 1u << FA_AN : 0u) | (mismatch ? 1u << FA_MIS : 0u) | (barrier ? 0u : 1u << FA_ROUND);
    if (!barrier) { acc.best_rng = tmx - tmn; acc.best_k = seq0 + j; }
  }
}

// Folds a warp's totals: counters into the CTA's shared counters, per-position bandwidth sums and the Eq. 2
// candidate into the warp's row of `sh`.
template <int L>
__device__ __forceinline__ void warp_fold(FastAcc& acc, double (&bw)[8], u32 n, FusedShared& sh) {
  constexpr int GW = 32 / L;
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const u32 n_comp = __reduce_add_sync(FULLM, (acc.groups >> FA_COMP) & 63u), n_bar = __reduce_add_sync(FULLM, (acc.groups >> FA_BAR) & 63u),
            n_an = __reduce_add_sync(FULLM, (acc.groups >> FA_AN) & 63u), n_mis = __reduce_add_sync(FULLM, (acc.groups >> FA_MIS) & 63u),
            n_round = __reduce_add_sync(FULLM, acc.groups >> FA_ROUND), n_fs = __reduce_add_sync(FULLM, acc.flagged & 0xFFFFu),
            n_fd = __reduce_add_sync(FULLM, acc.flagged >> 16), n_def = __reduce_add_sync(FULLM, acc.n_def);
  u32 rng = acc.best_rng, bk = acc.best_k;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const u32 o_rng = __shfl_xor_sync(FULLM, rng, d), o_k = __shfl_xor_sync(FULLM, bk, d);
    if (o_k != NONE && (bk == NONE || o_rng > rng || (o_rng == rng && o_k < bk))) { rng = o_rng; bk = o_k; }
  }
  if (L == 1) {
    const double tot = warp_sum8(bw, lane);                  // lane l holds member 4 bit4(l) + 2 bit3(l) + bit2(l)
    if ((lane & 3) == 0) sh.bw[wid][lane >> 2] = tot;
  } else {
    // sums over the warp's groups: each round halves the values a lane carries
    const u32 p0 = (lane % L) * 8;
    u32 off = 0;
#pragma unroll
    for (int bit = 16, w = 4; bit >= L; bit >>= 1, w >>= 1) {
      const bool hi = (lane & bit) != 0;
#pragma unroll
      for (int i = 0; i < w; ++i) {
        const double send = hi ? bw[i] : bw[i + w], keep = hi ? bw[i + w] : bw[i];
        bw[i] = keep + __shfl_xor_sync(FULLM, send, bit);
      }
      off += hi ? (u32)w : 0u;
    }
#pragma unroll
    for (int i = 0; i < 8 / GW; ++i) sh.bw[wid][p0 + off + i] = bw[i];
  }
  if (lane == 0) {
    sh.rounds[wid] = n_round; sh.n_an[wid] = n_an; sh.n_def[wid] = n_def; sh.brng[wid] = rng; sh.bk[wid] = bk;
    if (n_comp) { atomicAdd(&sh.cnt[SC_COMP], n_comp); atomicAdd(&sh.cnt[SC_PRES], n_comp * n); }
    if (n_bar) atomicAdd(&sh.cnt[SC_BAR], n_bar);
    if (n_an) atomicAdd(&sh.cnt[SC_AN], n_an);
    if (n_mis) atomicAdd(&sh.cnt[SC_MIS], n_mis);
    if (n_fs) atomicAdd(&sh.cnt[SC_FS], n_fs);
    if (n_fd) atomicAdd(&sh.cnt[SC_FD], n_fd);
  }
}

__device__ __forceinline__ void flush_counters(const WinDesc& D, const FusedShared& sh) {
  count_add(D.counters, C_COMPLETE, sh.cnt[SC_COMP]); count_add(D.counters, C_BARRIER, sh.cnt[SC_BAR]); count_add(D.counters, C_ANALYSED, sh.cnt[SC_AN]);
  count_add(D.counters, C_MISMATCH, sh.cnt[SC_MIS]); count_add(D.counters, C_PRESENT, sh.cnt[SC_PRES]);
  count_add(D.counters, C_FLAG_SKEW, sh.cnt[SC_FS]); count_add(D.counters, C_FLAG_DUR, sh.cnt[SC_FD]);
}

// Class-0 CTA (n <= 8): up to FUSED_WT_PER_CTA warp-tiles of one window and one time chunk, each up to 32 consecutive op
// counters of one communicator with its own summary entry. A warp takes every eighth tile and meets the other warps
// only at the end, so the warps of a CTA drift apart and one warp's gathers overlap another's arithmetic.
__device__ __forceinline__ void fused_small_cta(const WinDesc& D, const FusedCta& t, const WarpTile* __restrict__ wts, TileSum* __restrict__ sums,
                                                const Registry& R, const Params& P, const DeferList& DL, FusedShared& sh) {
  const u32 wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                                          // the CTA's counters are zero
  for (u32 i = wid; i < t.wt_count; i += SMALL_SEQS / 32) {
    const WarpTile wt = wts[t.wt_first + i];
    FastAcc acc; double bw[8];
    if (wt.row.n == SMALL_N) fast_groups<1, true>(D, t.w, wt.row, R.members + wt.moff, wt.seq_off, wt.count, R, P, DL, sh, acc, bw);
    else fast_groups<1, false>(D, t.w, wt.row, R.members + wt.moff, wt.seq_off, wt.count, R, P, DL, sh, acc, bw);
    warp_fold<1>(acc, bw, wt.row.n, sh);
    __syncwarp();
    if (lane == 0) {
      TileSum ts; ts.best_rng = sh.brng[wid]; ts.best_k = sh.bk[wid]; ts.n_rounds = sh.rounds[wid]; ts.n_an = sh.n_an[wid]; ts.pad = sh.n_def[wid];
      sums[wt.sum_idx] = ts;
    }
    // per-rank bandwidth of the tile: lane m < n adds member m's sum
    const u32 rounds = sh.rounds[wid];
    if (lane < wt.row.n && rounds) {
      const u32 rank = R.members[wt.moff + lane];
      atomicAdd(&R.bw_sum[rank], sh.bw[wid][lane]); atomicAdd(&R.bw_cnt[rank], rounds);
    }
    __syncwarp();
  }
  __syncthreads();
  if (threadIdx.x == 0) flush_counters(D, sh);
}

// Class-1 CTA (9 <= n <= 128): one tile of 2048 / n_pad consecutive op counters of one communicator, 32 / L per warp;
// one summary entry.
template <int L>
__device__ __forceinline__ void fused_sub_cta(const WinDesc& D, const FusedCta& t, TileSum* __restrict__ sums, const Registry& R, const Params& P,
                                              const DeferList& DL, FusedShared& sh) {
  constexpr u32 GW = 32 / L, NW = SMALL_SEQS / 32;
  const u32 wid = threadIdx.x >> 5, n = t.row.n;
  const u32 first = wid * GW;
  const u32 cnt = first < t.count ? (t.count - first < GW ? t.count - first : GW) : 0u;
  FastAcc acc; double bw[8];
  if (L >= 8) {
    // the tile's records are gathered with lanes along the op counter and wait in shared memory as 32-bit keys
    if (threadIdx.x < 32) sh.t_bits[threadIdx.x] = 0;
    __syncthreads();
    stage_tile<L>(D, t.row, t.seq_off, t.count, sh);
    __syncthreads();
    if (n == (u32)(L * 8)) fast_groups<L, true, true>(D, t.w, t.row, R.members + t.moff, t.seq_off + first, cnt, R, P, DL, sh, acc, bw, first);
    else fast_groups<L, false, true>(D, t.w, t.row, R.members + t.moff, t.seq_off + first, cnt, R, P, DL, sh, acc, bw, first);
  } else if (n == (u32)(L * 8)) fast_groups<L, true>(D, t.w, t.row, R.members + t.moff, t.seq_off + first, cnt, R, P, DL, sh, acc, bw);
  else fast_groups<L, false>(D, t.w, t.row, R.members + t.moff, t.seq_off + first, cnt, R, P, DL, sh, acc, bw);
  warp_fold<L>(acc, bw, n, sh);
  __syncthreads();
  u32 rounds = 0;
#pragma unroll
  for (u32 q = 0; q < NW; ++q) rounds += sh.rounds[q];
  if (rounds) {
    const u32* mem = R.members + t.moff;
    for (u32 p = threadIdx.x; p < n; p += SMALL_SEQS) {
      double v = 0.0;
#pragma unroll
      for (u32 q = 0; q < NW; ++q) v += sh.bw[q][p];
      atomicAdd(&R.bw_sum[mem[p]], v);
      atomicAdd(&R.bw_cnt[mem[p]], rounds);
    }
  }
  if (threadIdx.x == 0) {
    u64 brng = sh.brng[0]; u32 bk = sh.bk[0], n_an = sh.n_an[0], n_def = sh.n_def[0];
    for (u32 q = 1; q < NW; ++q) { best_merge(brng, bk, sh.brng[q], sh.bk[q]); n_an += sh.n_an[q]; n_def += sh.n_def[q]; }
    TileSum ts; ts.best_rng = brng; ts.best_k = bk; ts.n_rounds = rounds; ts.n_an = n_an; ts.pad = n_def;
    sums[t.sum_idx] = ts;
    flush_counters(D, sh);
  }
}

__global__ void __launch_bounds__(SMALL_SEQS, CCLD_FUSED_MIN_CTAS) k_reduce_fused(const WinDesc* __restrict__ wd, const FusedCta* __restrict__ ctas,
    const WarpTile* __restrict__ wts, TileSum* __restrict__ sums, Registry R, Params P, DeferList DL) {
  __shared__ FusedShared sh;
  const FusedCta t = ctas[blockIdx.x];
  const WinDesc& D = wd[t.w];
  if (threadIdx.x < SC_COUNT) sh.cnt[threadIdx.x] = 0;
  if (threadIdx.x == 0) { sh.out.flags = D.flags; sh.out.gi64 = D.gi64; sh.out.gu32 = D.gu32; sh.out.gbw = D.gbw; sh.out.G = D.n_groups; }
  if (t.cls == 0) { fused_small_cta(D, t, wts, sums, R, P, DL, sh); return; }
  __syncthreads();
  const u32 n_pad = mid_npad(t.row.n);
  if (n_pad == 32) fused_sub_cta<4>(D, t, sums, R, P, DL, sh);
  else if (n_pad == 64) fused_sub_cta<8>(D, t, sums, R, P, DL, sh);
  else fused_sub_cta<16>(D, t, sums, R, P, DL, sh);
}

// ------------------------------------------------------------------------------------------------
// the groups k_reduce_fused set aside: one warp per group, ring position p in lane p % 32; 64-bit
// throughout, order statistics by counting ranks (a group has at most 128 members)
// ------------------------------------------------------------------------------------------------
constexpr int DEF_WARPS = 4;
constexpr int DEF_GRID = 148 * 4;   // grid-stride over the list: four CTAs per SM of a B200
constexpr int DEF_Q = WARP_N / 32;

__device__ __forceinline__ u64 warp_max64(u64 v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) { const u64 o = shfl_xor64(v, d); v = o > v ? o : v; }
  return v;
}
__device__ __forceinline__ u64 warp_min64(u64 v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) { const u64 o = shfl_xor64(v, d); v = o < v ? o : v; }
  return v;
}
// k-th smallest (0-based) of x over positions < n: the element that k others precede in (value, position) order
__device__ __forceinline__ u64 rank_select(const u64 (&x)[DEF_Q], u32 n, u32 k, u64* key, u32 lane) {
  __syncwarp();
#pragma unroll
  for (int i = 0; i < DEF_Q; ++i) { const u32 p = lane + 32u * i; if (p < n) key[p] = x[i]; }
  __syncwarp();
  u64 res = 0; bool mine = false;
#pragma unroll
  for (int i = 0; i < DEF_Q; ++i) {
    const u32 p = lane + 32u * i;
    if (p < n) {
      u32 r = 0;
      for (u32 q = 0; q < n; ++q) { const u64 kq = key[q]; r += (kq < x[i] || (kq == x[i] && q < p)) ? 1u : 0u; }
      if (r == k) { mine = true; res = x[i]; }
    }
  }
  const u32 src = (u32)__ffs(__ballot_sync(FULLM, mine)) - 1u;
  return __shfl_sync(FULLM, res, src & 31);
}

__global__ void __launch_bounds__(DEF_WARPS * 32) k_reduce_deferred(const WinDesc* __restrict__ wd, DeferList DL, Registry R, Params P, i64 now) {
  __shared__ u64 s_key[DEF_WARPS][WARP_N];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u64* key = s_key[wid];
  const u32 total = *DL.count;
  for (u32 e = blockIdx.x * DEF_WARPS + wid; e < total; e += gridDim.x * DEF_WARPS) {
    const u64 ent = DL.entries[e];
    const WinDesc& D = wd[(u32)(ent >> 32)];
    const u64 g = (u32)ent;
    u32 c;
    { // owner: the last communicator whose first group is <= g
      u32 lo = 0, hi = R.n_comms - 1;
      while (lo < hi) { const u32 mid = (lo + hi + 1) >> 1; if (D.ranges[mid].group0 <= g) lo = mid; else hi = mid - 1; }
      c = lo;
    }
    const RangeRow row = D.ranges[c];
    const u32 n = row.n, so = (u32)(g - row.group0);
    const u32* mem = R.members + R.comm_moff[c];

    bool pres[DEF_Q]; i64 ta[DEF_Q], tb[DEF_Q]; u64 by[DEF_Q]; u32 op[DEF_Q], ch[DEF_Q];
    u32 npres = 0, first_p = NONE; bool miss = false, inflight = false, bad = false;
    i64 age = -1, x_max = INT64_MIN; u64 ck = 0;
#pragma unroll
    for (int i = 0; i < DEF_Q; ++i) {
      const u32 p = lane + 32u * i;
      pres[i] = false; ta[i] = 0; tb[i] = 0; by[i] = 0; op[i] = 0; ch[i] = 0;
      if (p < n) {
        const u32 idx = D.perm[perm_at(row, so, p)];
        if (idx == NONE) miss = true;
        else {
          pres[i] = true; ++npres; if (first_p == NONE) first_p = p;
          ta[i] = D.t_enter[idx]; tb[i] = D.t_exit[idx]; by[i] = D.bytes[idx]; op[i] = D.op[idx];
          if (D.send_chg != nullptr) { const u32 sc = D.send_chg[idx], rc = D.recv_chg[idx]; ch[i] = sc > rc ? sc : rc; }
          if (tb[i] == -1) { inflight = true; const i64 ag = now - ta[i]; age = ag > age ? ag : age; }
          else if (ta[i] < 0 || tb[i] < ta[i]) bad = true;
          x_max = tb[i] > x_max ? tb[i] : x_max;
          const u64 k2 = ((u64)ch[i] << 32) | (u64)(NONE - p);          // most changes, then the lowest position
          ck = k2 > ck ? k2 : ck;
        }
      }
    }
    npres = __reduce_add_sync(FULLM, npres); first_p = __reduce_min_sync(FULLM, first_p);
    miss = __any_sync(FULLM, miss); inflight = __any_sync(FULLM, inflight); bad = __any_sync(FULLM, bad);
    age = (i64)(warp_max64((u64)age ^ 0x8000000000000000ull) ^ 0x8000000000000000ull);
    x_max = (i64)(warp_max64((u64)x_max ^ 0x8000000000000000ull) ^ 0x8000000000000000ull);
    ck = warp_max64(ck);
    const bool complete = !miss && !inflight && !bad;
    // op set: the first present member's op and size
    const bool have_first = first_p != NONE;
    u64 gbytes = 0; u32 gop = 0;
    if (have_first) {
      u64 fby = 0; u32 fop = 0;
#pragma unroll
      for (int i = 0; i < DEF_Q; ++i) if ((first_p >> 5) == (u32)i) { fby = by[i]; fop = op[i]; }
      gbytes = __shfl_sync(FULLM, fby, first_p & 31); gop = __shfl_sync(FULLM, fop, first_p & 31);
    }
    bool mm = false;
#pragma unroll
    for (int i = 0; i < DEF_Q; ++i) if (pres[i] && (op[i] != gop || by[i] != gbytes)) mm = true;
    const bool mismatch = __any_sync(FULLM, mm);
    const bool barrier = have_first && gop == CCLD_OP_ALLREDUCE && gbytes < P.barrier_bytes;
    const bool analysed = complete && !barrier && n >= P.min_group;
    const bool hang = !complete && inflight && age > P.hang_ns && !barrier;
    const u32 gfl = (mismatch ? CCLD_G_OPSET_MISMATCH : 0) | (barrier ? CCLD_G_BARRIER : 0) | (inflight ? CCLD_G_INFLIGHT : 0) |
                    (bad ? CCLD_G_BAD_TIME : 0) | (complete ? CCLD_G_COMPLETE : CCLD_G_INCOMPLETE) | (analysed ? CCLD_G_ANALYSED : 0) |
                    (hang ? CCLD_G_HANG_ALERT : 0);

    u64 e_min = 0, e_max = 0, tmax = 0, tmin = 0, med_s = 0, mad_s = 0, med_d = 0, mad_d = 0; u32 pmax = 0, pmin = 0;
    u32 n_fs = 0, n_fd = 0;
    u32 fl[DEF_Q];
#pragma unroll
    for (int i = 0; i < DEF_Q; ++i) fl[i] = CCLD_F_NOT_ANALYSED | (pres[i] ? 0 : CCLD_F_MISSING);
    double num = 1.0, den = 1.0; bus_factor(gop, n, &num, &den);
    const double bn = (double)gbytes * num;
    if (complete) {
      u64 sk[DEF_Q], du[DEF_Q];
      u64 l_emin = U64_MAX_, l_emax = 0, l_tmax = 0, l_tmin = U64_MAX_;
#pragma unroll
      for (int i = 0; i < DEF_Q; ++i) {
        du[i] = (u64)(tb[i] - ta[i]);
        if (pres[i]) {
          const u64 te = (u64)ta[i];
          l_emin = te < l_emin ? te : l_emin; l_emax = te > l_emax ? te : l_emax;
          l_tmax = du[i] > l_tmax ? du[i] : l_tmax; l_tmin = du[i] < l_tmin ? du[i] : l_tmin;
        }
      }
      e_min = warp_min64(l_emin); e_max = warp_max64(l_emax); tmax = warp_max64(l_tmax); tmin = warp_min64(l_tmin);
      u32 c_mx = NONE, c_mn = NONE;                          // ties: the lowest position
#pragma unroll
      for (int i = DEF_Q - 1; i >= 0; --i) if (pres[i]) { const u32 p = lane + 32u * i; if (du[i] == tmax) c_mx = p; if (du[i] == tmin) c_mn = p; }
      pmax = __reduce_min_sync(FULLM, c_mx); pmin = __reduce_min_sync(FULLM, c_mn);
#pragma unroll
      for (int i = 0; i < DEF_Q; ++i) sk[i] = (u64)ta[i] - e_min;
      if (!barrier) {
#pragma unroll
        for (int i = 0; i < DEF_Q; ++i) if (pres[i]) { const u32 p = lane + 32u * i; atomicAdd(&R.bw_sum[mem[p]], busbw_fast(bn, den, (i64)du[i])); atomicAdd(&R.bw_cnt[mem[p]], 1u); }
      }
      if (analysed) {
        const u32 k = (n - 1) >> 1;
        u64 dv[DEF_Q];
        med_s = rank_select(sk, n, k, key, lane);
#pragma unroll
        for (int i = 0; i < DEF_Q; ++i) dv[i] = absdiff(sk[i], med_s);
        mad_s = rank_select(dv, n, k, key, lane);
        med_d = rank_select(du, n, k, key, lane);
#pragma unroll
        for (int i = 0; i < DEF_Q; ++i) dv[i] = absdiff(du[i], med_d);
        mad_d = rank_select(dv, n, k, key, lane);
#pragma unroll
        for (int i = 0; i < DEF_Q; ++i) {
          if (pres[i]) {
            const u32 p = lane + 32u * i;
            const bool so_ = mul_gt(absdiff(sk[i], med_s), 1000u, mad_s, P.k_milli), shi = sk[i] > med_s;
            const bool dq = mul_gt(absdiff(du[i], med_d), 1000u, mad_d, P.k_milli), dhi = du[i] > med_d;
            fl[i] = (so_ ? CCLD_F_SKEW_OUT : 0) | (dq ? CCLD_F_DUR_OUT : 0) | (shi ? CCLD_F_SKEW_HI : 0) | (dhi ? CCLD_F_DUR_HI : 0);
            if (so_) { ++n_fs; atomicAdd(&R.votes[(u64)mem[p] * 4 + (shi ? 0 : 1)], 1u); }
            if (dq) { ++n_fd; atomicAdd(&R.votes[(u64)mem[p] * 4 + (dhi ? 2 : 3)], 1u); }
          }
        }
      }
    }
    n_fs = __reduce_add_sync(FULLM, n_fs); n_fd = __reduce_add_sync(FULLM, n_fd);
    // ---- outputs ----
    {
      u8* __restrict__ fp = D.flags + row.slot0 + (u64)so * n;
#pragma unroll
      for (int i = 0; i < DEF_Q; ++i) { const u32 p = lane + 32u * i; if (p < n) fp[p] = (u8)fl[i]; }
    }
    if (lane == 0) {
      const u64 G = D.n_groups;
      const i64 span = complete ? x_max - (i64)e_min : 0;
      if (hang) raise_alert(D, R.comm_id[c], row.seq_lo + so, age);
      D.gi64[(u64)GI_E_MIN * G + g] = complete ? (i64)e_min : 0; D.gi64[(u64)GI_ARRIVAL_SKEW * G + g] = complete ? (i64)(e_max - e_min) : 0;
      D.gi64[(u64)GI_T_MAX * G + g] = (i64)tmax; D.gi64[(u64)GI_T_MIN * G + g] = (i64)tmin; D.gi64[(u64)GI_SPAN * G + g] = span;
      D.gi64[(u64)GI_MED_SKEW * G + g] = (i64)med_s; D.gi64[(u64)GI_MAD_SKEW * G + g] = (i64)mad_s;
      D.gi64[(u64)GI_MED_DUR * G + g] = (i64)med_d; D.gi64[(u64)GI_MAD_DUR * G + g] = (i64)mad_d;
      D.gu32[(u64)GU_RANK_TMIN * G + g] = complete ? mem[pmin] : 0; D.gu32[(u64)GU_RANK_TMAX * G + g] = complete ? mem[pmax] : 0;
      D.gu32[(u64)GU_MAX_CHG * G + g] = complete ? (u32)(ck >> 32) : 0;
      D.gu32[(u64)GU_RANK_MAX_CHG * G + g] = complete ? mem[NONE - (u32)ck] : 0;
      D.gu32[(u64)GU_N_PRESENT * G + g] = npres; D.gu32[(u64)GU_GFLAGS * G + g] = gfl;
      D.gbw[g] = complete ? busbw_fast(bn, den, span) : 0.0;
      count_add(D.counters, complete ? C_COMPLETE : C_INCOMPLETE, 1u);
      if (barrier) count_add(D.counters, C_BARRIER, 1u);
      if (analysed) count_add(D.counters, C_ANALYSED, 1u);
      if (mismatch) count_add(D.counters, C_MISMATCH, 1u);
      count_add(D.counters, C_PRESENT, npres); count_add(D.counters, C_FLAG_SKEW, n_fs); count_add(D.counters, C_FLAG_DUR, n_fd);
    }
  }
}

}  // namespace ccld
