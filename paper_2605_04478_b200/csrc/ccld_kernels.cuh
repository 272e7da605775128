// Kernels of the CCL-D analyzer hot path for sm_100a. Everything the analysis computes runs here;
// the host side only sizes buffers and launches.
//
//   k_seq_range     group-by, part 1: op-counter range per (window, communicator)
//   k_plan          group-by, part 2: closed-form slot layout (prefix sums over communicators),
//                   and the work list for the reduction kernels
//   k_slot_scatter  group-by, part 3: perm[slot] = record index
//   k_reduce_fused  per-op reductions + median/MAD + flags + votes for n <= 128, chunk-major work list:
//                   n <= 8 one thread per group (warp-tiles), 9 <= n <= 128 n_pad / 8 lanes per group (register /
//                   shuffle bitonic network); complete groups whose times fit 32-bit offsets
//   k_reduce_deferred  the groups k_reduce_fused sets aside (incomplete, in flight, 64-bit spreads)
//   k_reduce_mid    same, 129 <= n <= 1024 (shared-memory bitonic sort, several groups per CTA)
//   k_reduce_large  same, n > 1024 (ccld_large.cuh: a CTA per tile of 8 op counters, several groups side by side, radix select)
//   k_reduce_large_deferred  the groups k_reduce_large sets aside
//   k_window_rounds Eq. 2 per (communicator, window): round counts, selected round, location candidates
//   k_window_decide Eq. 1, 3, 4 per communicator, windows in order: baseline state, class, slow location
//   k_hang_locate   hang decision tree over presence / completion / progress counters
//   k_suspects, k_rank_sort_*  suspect list and ordered output lists
#pragma once
#include "ccld_device.cuh"

namespace ccld {

// ------------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 hash_home(const Registry& R, u32 id) { return (id * 2654435761u) & R.hash_mask; }

// Continues a probe sequence whose first entry (at the home slot) the caller already holds.
__device__ __forceinline__ uint4 comm_find(const Registry& R, u32 id, uint4 e) {
  u32 h = hash_home(R, id);
  for (u32 probe = 0; probe <= R.hash_mask; ++probe) {
    if (e.y == NONE || e.x == id) return e;
    h = (h + 1) & R.hash_mask;
    e = R.hash[h];
  }
  return make_uint4(0, NONE, 0, 0);
}

__device__ __forceinline__ u32 comm_lookup(const Registry& R, u32 id) { return comm_find(R, id, R.hash[hash_home(R, id)]).y; }

__device__ __forceinline__ u32 pos_lookup(const Registry& R, u32 rank, u32 c) {
  if (rank >= R.n_ranks) return NONE;
  u32 b = R.rank_ptr[rank], e = R.rank_ptr[rank + 1];
  for (u32 i = b; i < e; ++i)
    if (R.ent_comm[i] == c) return R.ent_pos[i];
  return NONE;
}

// a * ka > b * kb in exact 128-bit arithmetic
__device__ __forceinline__ bool mul_gt(u64 a, u32 ka, u64 b, u32 kb) {
  u64 alo = a * ka, ahi = __umul64hi(a, (u64)ka);
  u64 blo = b * kb, bhi = __umul64hi(b, (u64)kb);
  return ahi > bhi || (ahi == bhi && alo > blo);
}
__device__ __forceinline__ bool mul_lt(u64 a, u32 ka, u64 b, u32 kb) { return mul_gt(b, kb, a, ka); }

// bus-bandwidth factor num/den of an op over n ranks
__device__ __forceinline__ void bus_factor(u32 op, u32 n, double* num, double* den) {
  if (op == CCLD_OP_ALLREDUCE) { *num = 2.0 * (double)(n - 1); *den = (double)n; }
  else if (op == CCLD_OP_ALLGATHER || op == CCLD_OP_REDUCESCATTER || op == CCLD_OP_ALLTOALL) { *num = (double)(n - 1); *den = (double)n; }
  else { *num = 1.0; *den = 1.0; }
}
__device__ __forceinline__ double busbw(double bytes_num, double den, i64 t) {
  return t > 0 ? bytes_num / ((double)t * den) : 0.0;
}

__device__ __forceinline__ u64 absdiff(u64 a, u64 b) { return a >= b ? a - b : b - a; }

// Where the record index of (communicator row, op-counter offset, ring position) sits in `perm`. The permutation
// is member-major inside a communicator - [position][op counter] - so that consecutive records of one rank, which
// carry consecutive op counters, scatter to consecutive entries, and so that a warp reading 32 consecutive op
// counters of one member reads 128 contiguous bytes. Flags and per-op rows stay group-major.
__device__ __forceinline__ u64 perm_at(const RangeRow& row, u32 seq_off, u32 pos) { return row.slot0 + (u64)pos * row.n_seq + seq_off; }

__device__ __forceinline__ u64 shfl_xor64(u64 v, int m) { return __shfl_xor_sync(0xFFFFFFFFu, v, m); }

__device__ __forceinline__ void count_add(u64* counters, int which, u32 v) {
  if (v) atomicAdd((ull*)&counters[which], (ull)v);
}

__device__ __forceinline__ void raise_alert(const WinDesc& D, u32 comm_id, u32 seq, i64 age) {
  ull k = atomicAdd((ull*)&D.counters[C_ALERTS], 1ull);
  if (k < CCLD_MAX_ALERTS_PER_WINDOW) { ccld_hang_alert a; a.comm = comm_id; a.seq = seq; a.age_ns = age; D.alerts[k] = a; }
}

// Eq. 2 candidate merge: larger range wins, then the earlier op counter (k = NONE means "no round")
__device__ __forceinline__ void best_merge(u64& rng, u32& k, u64 o_rng, u32 o_k) {
  if (o_k != NONE && (k == NONE || o_rng > rng || (o_rng == rng && o_k < k))) { rng = o_rng; k = o_k; }
}
__device__ __forceinline__ void best_warp_reduce(u64& rng, u32& k) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const u64 o_rng = shfl_xor64(rng, d); const u32 o_k = __shfl_xor_sync(0xFFFFFFFFu, k, d);
    best_merge(rng, k, o_rng, o_k);
  }
}

// ------------------------------------------------------------------------------------------------
// record-streaming kernels (group-by parts 1 and 3). A CTA stages the key columns of REC_PER_CTA
// consecutive records in shared memory with coalesced 128-bit loads; each thread then walks a run of
// REC_RUN consecutive records. In rank-major or arrival-ordered uploads a run cycles through a handful
// of (rank, communicator) pairs, which the thread keeps in registers, so the registry is consulted a
// few times per run instead of once per record. Any order is handled: a full cache is flushed.
// ------------------------------------------------------------------------------------------------
constexpr int REC_RUN = REC_PER_CTA / REC_THREADS;       // consecutive records per thread
constexpr int REC_PITCH = REC_RUN + 1;                   // shared-memory pitch of a run (conflict-free walks)
constexpr int RC = 4;                                    // cached pairs per thread

// Copies n_valid <= REC_PER_CTA elements of a u32 column, starting at record `first`, into s[(i / RUN) * PITCH + i % RUN].
__device__ __forceinline__ void stage_column(const u32* __restrict__ col, u64 first, u32 n_valid, u32* s) {
  if ((((uintptr_t)(col + first)) & 15) == 0) {
    for (u32 q = threadIdx.x; q < REC_PER_CTA / 4; q += REC_THREADS) {
      const u32 i = q * 4;
      if (i + 4 <= n_valid) {
        const uint4 v = *reinterpret_cast<const uint4*>(col + first + i);
        u32* d = s + (i / REC_RUN) * REC_PITCH + (i % REC_RUN);      // REC_RUN is a multiple of 4: the four stay in one run
        d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
      } else {
        for (u32 k = i; k < n_valid; ++k) s[(k / REC_RUN) * REC_PITCH + (k % REC_RUN)] = col[first + k];
      }
    }
  } else {
    for (u32 i = threadIdx.x; i < n_valid; i += REC_THREADS) s[(i / REC_RUN) * REC_PITCH + (i % REC_RUN)] = col[first + i];
  }
}

__device__ __forceinline__ void range_widen(const WinDesc& D, u32 c, u32 mn, u32 mx) {
  if (mn < __ldcg(&D.rmin[c])) atomicMin(&D.rmin[c], mn);
  if (mx > __ldcg(&D.rmax[c])) atomicMax(&D.rmax[c], mx);
}

// A CTA keeps the op-counter extremes of every communicator it meets in a shared-memory table indexed by the
// communicator's registry index (registries of up to RANGE_DIRECT communicators; beyond that updates go to global
// memory, checked before each atomic) and merges the entries it touched into the window's global ranges at the end.
constexpr u32 RANGE_DIRECT = 4096;
inline size_t range_smem_bytes(u32 n_comms) { return n_comms <= RANGE_DIRECT ? (size_t)8 * n_comms : 0; }

__device__ __forceinline__ void range_put(const WinDesc& D, u32* s_mn, u32* s_mx, u32 c, u32 mn, u32 mx) {
  if (s_mn != nullptr) { atomicMin(&s_mn[c], mn); atomicMax(&s_mx[c], mx); }
  else range_widen(D, c, mn, mx);
}

// ---- group-by, part 1: which op counters does every communicator cover in every window ----
// A thread takes a run of REC_RUN consecutive records. A rank's stream alternates between a handful of communicators, so
// the thread folds its run in registers, one distinct communicator at a time (up to RANGE_FOLDS of them), and the warp
// then merges what its lanes found - in a rank-major upload all lanes meet the same few communicators - so that one lane
// updates the CTA's table per communicator. Records left over after the folds (an upload in arrival or random order)
// look their communicator up and update the table themselves: one registry lookup and two shared-memory atomics per
// record at worst.
constexpr int RANGE_FOLDS = 4;
constexpr int RANGE_WARP_FOLDS = 8;
constexpr u32 RANGE_BLOCKS_MAX = 16;                  // blocks of REC_PER_CTA records a CTA takes at most (the host takes fewer for small batches)

// cid[i] for the lowest i with bit i of `left` set (any element if left is 0)
__device__ __forceinline__ u32 first_left(const u32 (&cid)[REC_RUN], u32 left) {
  static_assert(REC_RUN == 16, "selection tree over a run of 16");
  const u32 b = (u32)__ffs(left) - 1u;
  u32 x8[8], x4[4];
#pragma unroll
  for (int i = 0; i < 8; ++i) x8[i] = (b & 8u) ? cid[8 + i] : cid[i];
#pragma unroll
  for (int i = 0; i < 4; ++i) x4[i] = (b & 4u) ? x8[4 + i] : x8[i];
  const u32 y0 = (b & 2u) ? x4[2] : x4[0], y1 = (b & 2u) ? x4[3] : x4[1];
  return (b & 1u) ? y1 : y0;
}

__global__ void __launch_bounds__(REC_THREADS) k_seq_range(const WinDesc* __restrict__ wd, Registry R, u32 blocks_per_cta) {
  extern __shared__ u32 s_dyn[];
  u32* const s_mn = R.n_comms <= RANGE_DIRECT ? s_dyn : nullptr;
  u32* const s_mx = R.n_comms <= RANGE_DIRECT ? s_dyn + R.n_comms : nullptr;
  const WinDesc& D = wd[blockIdx.y];                          // grid: (CTAs of the largest window, windows)
  if ((u64)blockIdx.x * blocks_per_cta * REC_PER_CTA >= D.n_rec) return;
  const u32 lane = threadIdx.x & 31;
  if (s_mn != nullptr) {
    for (u32 c = threadIdx.x; c < R.n_comms; c += REC_THREADS) { s_mn[c] = NONE; s_mx[c] = 0; }
    __syncthreads();
  }
  // a CTA takes blocks_per_cta consecutive blocks of the window, one after the other, and keeps one table for them: the
  // table's set-up, its barriers and its merge into the window's ranges are paid once
  for (u32 blk = 0; blk < blocks_per_cta; ++blk) {
    const u64 first = ((u64)blockIdx.x * blocks_per_cta + blk) * REC_PER_CTA;
    if (first >= D.n_rec) break;
    const u32 n_valid = D.n_rec - first < REC_PER_CTA ? (u32)(D.n_rec - first) : (u32)REC_PER_CTA;
    const u32 r0 = threadIdx.x * REC_RUN;
    const u32 len = r0 >= n_valid ? 0u : (n_valid - r0 < REC_RUN ? n_valid - r0 : (u32)REC_RUN);
    // the run goes straight into registers: four 128-bit loads per column where the column allows it
    u32 cid[REC_RUN], sq[REC_RUN];
    {
      const u32* __restrict__ pc = D.comm + first + r0; const u32* __restrict__ ps = D.seq + first + r0;
      if (len == REC_RUN && ((reinterpret_cast<uintptr_t>(pc) | reinterpret_cast<uintptr_t>(ps)) & 15) == 0) {
  #pragma unroll
        for (int q = 0; q < REC_RUN / 4; ++q) {
          const uint4 a = __ldg(reinterpret_cast<const uint4*>(pc) + q), b = __ldg(reinterpret_cast<const uint4*>(ps) + q);
          cid[4 * q] = a.x; cid[4 * q + 1] = a.y; cid[4 * q + 2] = a.z; cid[4 * q + 3] = a.w;
          sq[4 * q] = b.x; sq[4 * q + 1] = b.y; sq[4 * q + 2] = b.z; sq[4 * q + 3] = b.w;
        }
      } else {
  #pragma unroll
        for (int k = 0; k < REC_RUN; ++k) { cid[k] = (u32)k < len ? pc[k] : NONE; sq[k] = (u32)k < len ? ps[k] : 0u; }
      }
    }
    // records of the run not yet accounted for; a run cut short by the end of the window skips the folds (its padding
    // would match a record that names communicator 0xFFFFFFFF) and goes record by record
    const u32 tail = len < REC_RUN ? (1u << len) - 1u : 0u;
    u32 left = len < REC_RUN ? 0u : (1u << REC_RUN) - 1u;
    // warp folds: in a rank-major upload the 32 runs of a warp belong to one or two ranks, so all lanes meet the same few
    // communicators. One of them at a time - the communicator of the first record left in the lowest lane that has one -
    // is folded by every lane and reduced over the warp, and lane 0 updates the table once. The stage ends as soon as a
    // fold clears less than an eighth of what was left (an upload in another order): the lanes then fold on their own.
    {
      u32 remaining = __reduce_add_sync(0xFFFFFFFFu, (u32)__popc(left));
      for (int f = 0; f < RANGE_WARP_FOLDS && remaining != 0; ++f) {
        const u32 have = __ballot_sync(0xFFFFFFFFu, left != 0);
        const u32 id = __shfl_sync(0xFFFFFFFFu, first_left(cid, left), (u32)__ffs(have) - 1u);
        const uint4 h = comm_find(R, id, R.hash[hash_home(R, id)]);        // the same in every lane
        u32 m = 0, mn = NONE, mx = 0;
  #pragma unroll
        for (int k = 0; k < REC_RUN; ++k) {
          if (cid[k] == id) { m |= 1u << k; mn = min(mn, sq[k]); mx = max(mx, sq[k]); }
        }
        m &= left;                                             // a run cut short holds padding and takes no part
        u32 a = __reduce_min_sync(0xFFFFFFFFu, m ? mn : NONE), b = __reduce_max_sync(0xFFFFFFFFu, m ? mx : 0u);
        if (h.y != NONE && a < h.z) {
          // counters below the communicator's first name no operation: fold again without them
          mn = NONE; mx = 0;
  #pragma unroll
          for (int k = 0; k < REC_RUN; ++k) if (((m >> k) & 1u) && sq[k] >= h.z) { mn = min(mn, sq[k]); mx = max(mx, sq[k]); }
          a = __reduce_min_sync(0xFFFFFFFFu, mn); b = __reduce_max_sync(0xFFFFFFFFu, mx);
        }
        if (lane == 0 && h.y != NONE && a <= b) range_put(D, s_mn, s_mx, h.y, a, b);
        left &= ~m;
        const u32 cleared = __reduce_add_sync(0xFFFFFFFFu, (u32)__popc(m));
        const bool worth = cleared * 8u >= remaining;
        remaining -= cleared;
        if (!worth) break;
      }
    }
    // folds: the communicator of the first record still left takes every record of the run that names it
    for (int f = 0; f < RANGE_FOLDS && __any_sync(0xFFFFFFFFu, left != 0); ++f) {
      const bool act = left != 0;
      u32 id = NONE;
  #pragma unroll
      for (int k = REC_RUN - 1; k >= 0; --k) id = (left >> k) & 1u ? cid[k] : id;
      uint4 h = make_uint4(0, NONE, 0, 0);                      // (id, index, first counter, members); index NONE: unregistered
      if (act) h = comm_find(R, id, R.hash[hash_home(R, id)]);
      // a record folded earlier carries another id, so matching the id is enough (the run is complete: no padding)
      u32 m = 0, mn = NONE, mx = 0;
  #pragma unroll
      for (int k = 0; k < REC_RUN; ++k) {
        if (cid[k] == id) { m |= 1u << k; mn = min(mn, sq[k]); mx = max(mx, sq[k]); }
      }
      m &= left;
      if (h.y != NONE && m != 0 && mn < h.z) {
        // counters below the communicator's first name no operation: fold again without them
        mn = NONE; mx = 0;
  #pragma unroll
        for (int k = 0; k < REC_RUN; ++k) if (((m >> k) & 1u) && sq[k] >= h.z) { mn = min(mn, sq[k]); mx = max(mx, sq[k]); }
      }
      if (m == 0) { mn = NONE; mx = 0; }
      left &= ~m;
      // lanes that hold the same communicator merge: a few rounds, each led by the lowest lane still waiting
      bool mine = act && h.y != NONE && mn <= mx;
      u32 pend = __ballot_sync(0xFFFFFFFFu, mine);
      for (int it = 0; it < RANGE_FOLDS && pend; ++it) {
        const u32 leader = (u32)__ffs(pend) - 1u;
        const u32 lid = __shfl_sync(0xFFFFFFFFu, h.y, leader);
        const bool same = mine && h.y == lid;
        const u32 a = __reduce_min_sync(0xFFFFFFFFu, same ? mn : NONE), b = __reduce_max_sync(0xFFFFFFFFu, same ? mx : 0u);
        if (lane == leader) range_put(D, s_mn, s_mx, lid, a, b);
        if (same) mine = false;
        pend &= ~__ballot_sync(0xFFFFFFFFu, same);
      }
      if (mine) range_put(D, s_mn, s_mx, h.y, mn, mx);
    }
    // every record still left: one lookup each, four in flight
    left |= tail;
    if (left != 0) {
  #pragma unroll
      for (int k0 = 0; k0 < REC_RUN; k0 += 4) {
        uint4 h[4]; bool need[4];
  #pragma unroll
        for (int q = 0; q < 4; ++q) {
          need[q] = ((left >> (k0 + q)) & 1u) != 0;
          h[q] = need[q] ? R.hash[hash_home(R, cid[k0 + q])] : make_uint4(0, NONE, 0, 0);
        }
  #pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!need[q]) continue;
          const uint4 e = comm_find(R, cid[k0 + q], h[q]);
          if (e.y != NONE && sq[k0 + q] >= e.z) range_put(D, s_mn, s_mx, e.y, sq[k0 + q], sq[k0 + q]);
        }
      }
    }
  }
  if (s_mn == nullptr) return;
  __syncthreads();
  for (u32 c = threadIdx.x; c < R.n_comms; c += REC_THREADS) {
    const u32 mn = s_mn[c];
    if (mn != NONE) { atomicMin(&D.rmin[c], mn); atomicMax(&D.rmax[c], s_mx[c]); }      // nothing waits for these
  }
}

// ------------------------------------------------------------------------------------------------
// group-by, part 2: closed-form layout and work lists. One CTA per window scans the communicators.
//   slot(comm, seq, pos) = slot0[comm] + (seq - seq_lo[comm]) * n[comm] + pos
// ------------------------------------------------------------------------------------------------
struct PlanAcc { u64 groups, slots; u32 rows, t2, t3, pad; };

__device__ __forceinline__ PlanAcc plan_add(const PlanAcc& a, const PlanAcc& b) {
  PlanAcc r; r.groups = a.groups + b.groups; r.slots = a.slots + b.slots; r.rows = a.rows + b.rows;
  r.t2 = a.t2 + b.t2; r.t3 = a.t3 + b.t3; r.pad = 0; return r;
}
__device__ __forceinline__ PlanAcc plan_shfl_up(const PlanAcc& a, int d) {
  PlanAcc r;
  r.groups = __shfl_up_sync(0xFFFFFFFFu, a.groups, d); r.slots = __shfl_up_sync(0xFFFFFFFFu, a.slots, d);
  r.rows = __shfl_up_sync(0xFFFFFFFFu, a.rows, d); r.t2 = __shfl_up_sync(0xFFFFFFFFu, a.t2, d);
  r.t3 = __shfl_up_sync(0xFFFFFFFFu, a.t3, d); r.pad = 0;
  return r;
}

// op counters communicator c covers in the window (0 if none; clamped to 2^32 - 1)
__device__ __forceinline__ u32 plan_nseq(const WinDesc& D, const Registry& R, u32 c) {
  if (c >= R.n_comms) return 0;
  const u32 lo = D.rmin[c], hi = D.rmax[c];
  if (!(lo <= hi && lo != NONE)) return 0;
  const u64 ns = (u64)hi - lo + 1;
  return ns > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)ns;
}

__device__ __forceinline__ PlanAcc plan_item(const WinDesc& D, const Registry& R, u32 c) {
  PlanAcc a = {0, 0, 0, 0, 0, 0};
  const u32 ns = plan_nseq(D, R, c);
  if (ns) {
    const u32 n = R.comm_n[c], cls = comm_class(n);
    a.groups = ns; a.slots = (u64)ns * n; a.rows = 1;
    const u32 t = ceil_div(ns, tile_seqs(n));
    a.t2 = cls == 2 ? t : 0; a.t3 = cls == 3 ? t : 0;
  }
  return a;
}

// Exclusive prefix of `v` over the CTA's threads plus the CTA total, for PLAN_THREADS = 1024.
constexpr int PLAN_THREADS = 1024;
__device__ PlanAcc plan_block_scan(PlanAcc v, PlanAcc* total, PlanAcc* s_warp /*[33]*/) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  PlanAcc inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) { PlanAcc o = plan_shfl_up(inc, d); if (lane >= (u32)d) inc = plan_add(inc, o); }
  if (lane == 31) s_warp[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    PlanAcc x = s_warp[lane], xi = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { PlanAcc o = plan_shfl_up(xi, d); if (lane >= (u32)d) xi = plan_add(xi, o); }
    PlanAcc ex = plan_shfl_up(xi, 1);
    if (lane == 0) ex = PlanAcc{0, 0, 0, 0, 0, 0};
    s_warp[lane] = ex;
    if (lane == 31) s_warp[32] = xi;
  }
  __syncthreads();
  PlanAcc ex = plan_shfl_up(inc, 1);
  if (lane == 0) ex = PlanAcc{0, 0, 0, 0, 0, 0};
  PlanAcc r = plan_add(s_warp[wid], ex);
  *total = s_warp[32];
  __syncthreads();
  return r;
}

// The same for a pair of 32-bit counters.
__device__ uint2 plan_scan2(uint2 v, uint2* total, uint2* s_pair /*[33]*/) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  uint2 inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const u32 ox = __shfl_up_sync(0xFFFFFFFFu, inc.x, d), oy = __shfl_up_sync(0xFFFFFFFFu, inc.y, d);
    if (lane >= (u32)d) { inc.x += ox; inc.y += oy; }
  }
  if (lane == 31) s_pair[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    const uint2 x = s_pair[lane]; uint2 xi = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const u32 ox = __shfl_up_sync(0xFFFFFFFFu, xi.x, d), oy = __shfl_up_sync(0xFFFFFFFFu, xi.y, d);
      if (lane >= (u32)d) { xi.x += ox; xi.y += oy; }
    }
    s_pair[lane] = make_uint2(xi.x - x.x, xi.y - x.y);
    if (lane == 31) s_pair[32] = xi;
  }
  __syncthreads();
  const uint2 r = make_uint2(s_pair[wid].x + inc.x - v.x, s_pair[wid].y + inc.y - v.y);
  *total = s_pair[32];
  __syncthreads();
  return r;
}

// Work units (warp-tiles of class 0, CTA tiles of class 1) of communicator c in chunk tau; 0 for other classes.
__device__ __forceinline__ u32 chunk_units(u32 ns, u32 n, u32 T, u32 tau) {
  if (ns == 0 || comm_class(n) > 1) return 0;
  return ceil_div(chunk_size(ns, T, tau), tile_seqs(n));
}
// All units of communicator c in the window (its TileSum entries): full chunks plus the last one.
__device__ __forceinline__ u32 comm_units(u32 ns, u32 n, u32 T) {
  if (ns == 0 || comm_class(n) > 1) return 0;
  const u32 S = chunk_len(ns, T), nch = ceil_div(ns, S), U = tile_seqs(n);
  return (nch - 1) * ceil_div(S, U) + ceil_div(ns - (nch - 1) * S, U);
}

struct PlanLists { FusedCta* fcta; WarpTile* fwt; Tile* t2; Tile* t3; };

// A window that is given up leaves no work behind: zero ranges and scatter rows, zero totals.
__device__ __forceinline__ void plan_clear_rows(WinDesc& D, const Registry& R) {
  for (u32 c = threadIdx.x; c < R.n_comms; c += PLAN_THREADS) { RangeRow z = {0, 0, 0, R.comm_n[c], 0, 0, 0, 0}; D.ranges[c] = z; D.srow[c] = make_uint4(0, 0, 0, 0); }
  for (u64 i = threadIdx.x; i < (u64)R.n_ranks * RANK_TAB_K; i += PLAN_THREADS) D.rent[i] = make_uint4(0, 0, 0, 0);
}
__device__ __forceinline__ void plan_give_up(WinDesc& D, const Registry& R, u64 why) {
  plan_clear_rows(D, R);
  if (threadIdx.x == 0) {
    for (int q = 0; q < T_COUNT; ++q) D.totals[q] = 0;
    D.totals[T_FAILED] = why; D.totals[T_CHUNKS] = 1;
  }
}

// emit == 0: ranges, scatter rows and totals (the window is refused if it needs more than slot_cap slots).
// emit == 1: the work lists (base[] filled by the host from the totals).
// When the host sized the results from totals it expected (D.expect) instead of waiting for these, a window whose totals
// differ gives up and raises the poison flag; so does every window planned after the flag went up - in the same batch
// (seen here at emit == 1) or in a later one - so that windows are never analysed out of order. A window that gave up
// fills its stretch of the work lists with entries that hold no work, because the kernels that follow are launched
// over the expected lengths.
__global__ void __launch_bounds__(PLAN_THREADS) k_plan(WinDesc* __restrict__ wd, Registry R, PlanLists L, int emit) {
  __shared__ PlanAcc s_warp[33];
  __shared__ uint2 s_pair[33];
  __shared__ u32 s_red[32];
  __shared__ int s_failed;
  WinDesc& D = wd[blockIdx.x];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (emit) {
    if (D.expect != nullptr) {
      if (!D.totals[T_FAILED] && *(volatile u32*)D.poison != 0) { __syncthreads(); plan_give_up(D, R, FAILED_EXPECT); __syncthreads(); }
      if (D.totals[T_FAILED]) {
        const u64 n_cta = D.expect[T_FCTA], n2 = D.expect[T_TILES2], n3 = D.expect[T_TILES3];
        for (u64 j = threadIdx.x; j < n_cta; j += PLAN_THREADS) {
          FusedCta x; x.w = blockIdx.x; x.cls = 0; x.c = 0; x.seq_off = 0; x.count = 0; x.sum_idx = 0; x.wt_first = 0; x.wt_count = 0; x.moff = 0;
          x.row = RangeRow{0, 0, 0, 0, 0, 0, 0, 0};
          L.fcta[D.base[B_FCTA] + j] = x;
        }
        for (u64 j = threadIdx.x; j < n2; j += PLAN_THREADS) { Tile t; t.w = blockIdx.x; t.c = 0; t.seq_off = 0; t.count = 0; L.t2[D.base[B_T2] + j] = t; }
        for (u64 j = threadIdx.x; j < n3; j += PLAN_THREADS) { Tile t; t.w = blockIdx.x; t.c = 0; t.seq_off = 0; t.count = 0; L.t3[D.base[B_T3] + j] = t; }
        return;
      }
    } else if (D.totals[T_FAILED]) return;
  }

  if (!emit) {
    // 1. layout: groups, slots, rows; tiles of the two big classes; busiest fused-class communicator
    PlanAcc run = {0, 0, 0, 0, 0, 0};
    u32 mx = 0;
    for (u32 c0 = 0; c0 < R.n_comms; c0 += PLAN_THREADS) {
      const u32 c = c0 + threadIdx.x;
      PlanAcc it = plan_item(D, R, c), tot;
      PlanAcc ex = plan_add(run, plan_block_scan(it, &tot, s_warp));
      if (c < R.n_comms) {
        RangeRow r;
        r.seq_lo = it.rows ? D.rmin[c] : 0; r.n_seq = (u32)it.groups; r.row_idx = ex.rows; r.n = R.comm_n[c];
        r.group0 = ex.groups; r.slot0 = ex.slots; r.tile0 = 0; r.n_units = 0;
        D.ranges[c] = r;
        D.srow[c] = make_uint4((u32)r.slot0, (u32)(r.slot0 >> 32), r.n_seq, r.seq_lo);
        if (it.rows && comm_class(r.n) <= 1) mx = r.n_seq > mx ? r.n_seq : mx;
      }
      run = plan_add(run, tot);
    }
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    if (lane == 0) s_red[wid] = mx;
    __syncthreads();
    mx = 0;
    for (int q = 0; q < PLAN_THREADS / 32; ++q) mx = s_red[q] > mx ? s_red[q] : mx;
    u32 T = mx ? ceil_div(mx, CHUNK_REF) : 1u;
    T = T > CHUNK_MAX ? CHUNK_MAX : T;
    __syncthreads();
    // 2. summary entries of the fused classes
    u32 urun = 0;
    for (u32 c0 = 0; c0 < R.n_comms; c0 += PLAN_THREADS) {
      const u32 c = c0 + threadIdx.x;
      const u32 ns = plan_nseq(D, R, c), n = c < R.n_comms ? R.comm_n[c] : 1u;
      const u32 u = comm_units(ns, n, T);
      uint2 tot; const uint2 ex = plan_scan2(make_uint2(u, 0), &tot, s_pair);
      if (c < R.n_comms && u) { D.ranges[c].tile0 = urun + ex.x; D.ranges[c].n_units = u; }
      urun += tot.x;
    }
    // 3. CTAs and warp-tiles of the fused kernel, chunk by chunk
    u64 n_cta = 0, n_wt = 0;
    for (u32 tau = 0; tau < T; ++tau) {
      u32 wt = 0, c1 = 0;
      for (u32 c = threadIdx.x; c < R.n_comms; c += PLAN_THREADS) {
        const u32 n = R.comm_n[c], u = chunk_units(plan_nseq(D, R, c), n, T, tau);
        if (comm_class(n) == 0) wt += u; else c1 += u;
      }
      uint2 tot; plan_scan2(make_uint2(wt, c1), &tot, s_pair);
      n_cta += ceil_div(tot.x, FUSED_WT_PER_CTA) + tot.y; n_wt += tot.x;
    }
    if (threadIdx.x == 0) {
      // op counters further apart than 2^31, or more slots than the cap: refuse the window
      u64 failed = (run.slots > D.slot_cap || run.groups > 0x7FFFFFFFull || n_cta > 0x7FFFFFFFull || n_wt > 0x7FFFFFFFull) ? FAILED_CAPACITY : 0;
      if (!failed && D.expect != nullptr) {
        const u64* e = D.expect;
        const bool same = e[T_GROUPS] == run.groups && e[T_SLOTS] == run.slots && e[T_FCTA] == n_cta && e[T_FWT] == n_wt && e[T_FSUM] == urun &&
                          e[T_TILES2] == run.t2 && e[T_TILES3] == run.t3 && e[T_ROWS] == run.rows && e[T_CHUNKS] == T;
        if (!same || *(volatile u32*)D.poison != 0) { failed = FAILED_EXPECT; atomicExch(D.poison, 1u); }
      }
      s_failed = failed != 0;
      D.totals[T_GROUPS] = failed ? 0 : run.groups; D.totals[T_SLOTS] = failed ? 0 : run.slots;
      D.totals[T_FCTA] = failed ? 0 : n_cta; D.totals[T_FWT] = failed ? 0 : n_wt; D.totals[T_FSUM] = failed ? 0 : urun;
      D.totals[T_TILES2] = failed ? 0 : run.t2; D.totals[T_TILES3] = failed ? 0 : run.t3;
      D.totals[T_ROWS] = failed ? 0 : run.rows; D.totals[T_FAILED] = failed; D.totals[T_CHUNKS] = T;
      if (failed == FAILED_CAPACITY) atomicOr((unsigned*)&D.counters[C_ERR], (unsigned)CCLD_E_CAPACITY);
    }
    __syncthreads();
    if (s_failed) { plan_clear_rows(D, R); return; }
    // 4. every rank's inline (communicator, position) pairs resolved against this window's scatter rows, so that the
    //    scatter pass finds (op counters covered, first op counter, first slot of the member's column) with one load.
    //    Only where slots fit 32 bits and the member's whole column lies inside the table; other entries stay unused.
    if (run.slots <= 0xFFFFFFFFull) {
#pragma unroll 4
      for (u64 i = threadIdx.x; i < (u64)R.n_ranks * 2; i += PLAN_THREADS) {
        const uint4 t = R.rank_tab[i];
        uint4 e[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const u32 id = h ? t.z : t.x, cp = h ? t.w : t.y;
          if (id != NONE && cp != NONE && cp != RANK_TAB_OVERFLOW) {
            const uint4 sr = D.srow[cp >> RANK_TAB_POS_BITS];
            const u64 b = ((u64)sr.x | ((u64)sr.y << 32)) + (u64)(cp & ((1u << RANK_TAB_POS_BITS) - 1)) * sr.z;
            if (sr.z != 0 && b + sr.z <= run.slots) e[h] = make_uint4(id, sr.z, sr.w, (u32)b);
          }
        }
        D.rent[i * 2] = e[0]; D.rent[i * 2 + 1] = e[1];
      }
    }
    return;
  }

  // ---- emit ----
  const u32 T = (u32)D.totals[T_CHUNKS];
  // tiles of classes 2 and 3, communicator by communicator; summary indices of every communicator become batch-wide
  {
    PlanAcc run = {0, 0, 0, 0, 0, 0};
    for (u32 c0 = 0; c0 < R.n_comms; c0 += PLAN_THREADS) {
      const u32 c = c0 + threadIdx.x;
      PlanAcc it = plan_item(D, R, c), tot;
      PlanAcc ex = plan_add(run, plan_block_scan(it, &tot, s_warp));
      if (c < R.n_comms && it.rows) {
        const u32 n = R.comm_n[c], S = tile_seqs(n), cls = comm_class(n);
        if (cls <= 1) D.ranges[c].tile0 += D.base[B_FSUM];
        else {
          const u32 first = cls == 2 ? D.base[B_T2] + ex.t2 : D.base[B_T3] + ex.t3, nt = cls == 2 ? it.t2 : it.t3;
          Tile* dst = (cls == 2 ? L.t2 : L.t3) + first;
          D.ranges[c].tile0 = first; D.ranges[c].n_units = nt;
          for (u32 k = 0; k < nt; ++k) {
            Tile t; t.w = blockIdx.x; t.c = c; t.seq_off = k * S;
            const u64 left = it.groups - (u64)k * S; t.count = left < S ? (u32)left : S;
            dst[k] = t;
          }
        }
      }
      run = plan_add(run, tot);
    }
  }
  __syncthreads();
  // fused classes: chunk-major list of CTAs; a class-0 CTA takes eight consecutive warp-tiles
  u32 cta_base = D.base[B_FCTA], wt_base = D.base[B_FWT];
  for (u32 tau = 0; tau < T; ++tau) {
    u32 wt_run = 0, c1_run = 0;
    // class-1 CTAs come after the chunk's class-0 CTAs, whose number needs the chunk's warp-tile total first
    u32 wt_total = 0;
    {
      u32 wt = 0;
      for (u32 c = threadIdx.x; c < R.n_comms; c += PLAN_THREADS) { const u32 n = R.comm_n[c]; if (comm_class(n) == 0) wt += chunk_units(plan_nseq(D, R, c), n, T, tau); }
      uint2 tot; plan_scan2(make_uint2(wt, 0), &tot, s_pair);
      wt_total = tot.x;
    }
    const u32 n0 = ceil_div(wt_total, FUSED_WT_PER_CTA);
    for (u32 c0 = 0; c0 < R.n_comms; c0 += PLAN_THREADS) {
      const u32 c = c0 + threadIdx.x;
      const u32 ns = plan_nseq(D, R, c), n = c < R.n_comms ? R.comm_n[c] : 1u, cls = comm_class(n);
      const u32 u = chunk_units(ns, n, T, tau);
      uint2 tot; const uint2 ex = plan_scan2(make_uint2(cls == 0 ? u : 0, cls == 1 ? u : 0), &tot, s_pair);
      if (u) {
        const u32 S = chunk_len(ns, T), U = tile_seqs(n), cnt = chunk_size(ns, T, tau);
        const RangeRow crow = D.ranges[c]; const u64 cmoff = R.comm_moff[c];
        const u32 sum0 = crow.tile0 + tau * ceil_div(S, U);
        for (u32 k = 0; k < u; ++k) {
          const u32 off = tau * S + k * U, len = cnt - k * U < U ? cnt - k * U : U;
          if (cls == 0) { WarpTile x; x.c = c; x.seq_off = off; x.count = len; x.sum_idx = sum0 + k; x.row = crow; x.moff = cmoff; L.fwt[wt_base + wt_run + ex.x + k] = x; }
          else { FusedCta x; x.w = blockIdx.x; x.cls = 1; x.c = c; x.seq_off = off; x.count = len; x.sum_idx = sum0 + k; x.wt_first = 0; x.wt_count = 0;
                 x.row = crow; x.moff = cmoff; L.fcta[cta_base + n0 + c1_run + ex.y + k] = x; }
        }
      }
      wt_run += tot.x; c1_run += tot.y;
    }
    for (u32 j = threadIdx.x; j < n0; j += PLAN_THREADS) {
      FusedCta x; x.w = blockIdx.x; x.cls = 0; x.c = 0; x.seq_off = 0; x.count = 0; x.sum_idx = 0; x.moff = 0;
      x.row = RangeRow{0, 0, 0, 0, 0, 0, 0, 0};
      x.wt_first = wt_base + FUSED_WT_PER_CTA * j; x.wt_count = wt_total - FUSED_WT_PER_CTA * j < FUSED_WT_PER_CTA ? wt_total - FUSED_WT_PER_CTA * j : FUSED_WT_PER_CTA;
      L.fcta[cta_base + j] = x;
    }
    cta_base += n0 + c1_run; wt_base += wt_total;
  }
}

// ------------------------------------------------------------------------------------------------
// group-by, part 3: every accepted record drops its index into its slot. Two dependent loads per
// record in the common case - the rank's inline (communicator, index, position) pairs, then the
// communicator's scatter row - issued for four records at a time.
// ------------------------------------------------------------------------------------------------
// Registry walk for a record whose (rank, communicator) pair is not inline: returns index << 13 | position in the
// low word, or NONE there with the rejecting CCLD_E_* bit in the high word.
constexpr int SCAT_THREADS = 256;     // lanes on consecutive records: the stores of a warp land close together
constexpr int SCAT_PER_THREAD = 12;    // records per thread: enough to spread the two dependent table reads a warp starts with
constexpr int SCAT_PER_CTA = SCAT_THREADS * SCAT_PER_THREAD;
constexpr u32 SCAT_BLOCKS_MAX = 8;    // blocks of SCAT_PER_CTA records a CTA takes at most

__device__ __noinline__ u64 resolve_slow(const Registry& R, u32 rank, u32 cid) {
  const u32 c = comm_lookup(R, cid);
  if (c == NONE) return ((u64)CCLD_E_UNKNOWN_COMM << 32) | NONE;
  const u32 pos = pos_lookup(R, rank, c);
  if (pos == NONE) return ((u64)CCLD_E_NOT_MEMBER << 32) | NONE;
  return (c << RANK_TAB_POS_BITS) | pos;
}

// Where the record (rank, communicator id, op counter) goes, given the communicator's index c, the member's position
// and the scatter row of c. Returns false if nothing is stored; *err / *rej / *internal collect what went wrong.
__device__ __forceinline__ bool scatter_slot(const Registry& R, u32 c, u32 ns, u32 lo, u64 base_pos, u32 sq, u64 n_slots, u64* slot,
                                             u32* err, u32* rej, u32* internal) {
  if (ns == 0 || sq < lo) {
    if (sq < R.comm_seq0[c]) { *err |= CCLD_E_SEQ_RANGE; ++*rej; }
    else if (ns != 0) *internal = 1;
    return false;
  }
  *slot = base_pos + (sq - lo);
  if (sq - lo >= ns || *slot >= n_slots) { *internal = 1; return false; }
  return true;
}

constexpr u32 SCAT_LOCAL = 8;     // ranks, counted from the rank of the CTA's first record, whose table rows a CTA resolves once

// A CTA's records mostly belong to a few neighbouring ranks (a rank-major upload: one or two), so each warp first copies
// the resolved inline pairs of SCAT_LOCAL ranks - communicator id -> (counters covered, first counter, slot of the member's
// first counter), which the layout pass wrote for this window - into shared memory; a record of those ranks then needs no global table at all and, in windows of
// fewer than 2^32 slots, only 32-bit arithmetic. Any other record (another rank, a communicator beyond the inline pairs,
// a counter outside the range, a rejected record) takes the two dependent table loads and the full checks.
__global__ void __launch_bounds__(SCAT_THREADS, 4) k_slot_scatter(const WinDesc* __restrict__ wd, Registry R, u32 blocks_per_cta) {
  // (communicator id, counters covered, first counter, first slot) per resolved pair; counters covered 0: unused. Every
  // warp keeps its own copy, so no warp waits for another; two copies, because the entries of the next block are written
  // while lanes may still read those of the current one.
  __shared__ uint4 s_ent_all[2][SCAT_THREADS / 32][SCAT_LOCAL * RANK_TAB_K];
  static_assert(SCAT_LOCAL * RANK_TAB_K == 32, "one resolved pair per lane");
  const WinDesc& D = wd[blockIdx.y];                          // grid: (CTAs of the largest window, windows)
  const u64 base0 = (u64)blockIdx.x * blocks_per_cta * SCAT_PER_CTA;
  if (base0 >= D.n_rec) return;                               // (a window that was given up has empty scatter rows: nothing is stored)
  u32 err = 0, rej = 0, internal = 0;
  // descriptor fields in registers: the stores below could alias the descriptor as far as the compiler knows
  u32* const perm = D.perm; const u64 n_slots = D.n_slots; const uint4* const srow = D.srow; const u64 n_rec = D.n_rec;
  const uint4* const rent = D.rent;
  const u32 *c_rank = D.rank, *c_comm = D.comm, *c_seq = D.seq;
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  // the resolved pairs of the SCAT_LOCAL ranks that start at rank r_first, one per lane
  auto pairs_of = [&](u32 r_first) {
    const u32 r = r_first + lane / RANK_TAB_K;
    uint4 e = make_uint4(NONE, 0, 0, 0);
    if (r_first < R.n_ranks && r < R.n_ranks) e = rent[(u64)r * RANK_TAB_K + lane % RANK_TAB_K];
    return e;
  };
  // A CTA takes blocks_per_cta consecutive blocks. The chain "first record's rank -> that rank's resolved pairs" of a
  // block is started one block ahead, so a block waits for its records only.
  u32 r_first = c_rank[base0];
  uint4 e_mine = pairs_of(r_first);
  for (u32 blk = 0; blk < blocks_per_cta; ++blk) {
    const u64 base = base0 + (u64)blk * SCAT_PER_CTA;
    if (base >= n_rec) break;
    u32 rk[SCAT_PER_THREAD], cid[SCAT_PER_THREAD], sq[SCAT_PER_THREAD];
    u32 todo = 0;                                             // records that still need placing
#pragma unroll
    for (int k = 0; k < SCAT_PER_THREAD; ++k) {
      const u64 i = base + (u64)k * SCAT_THREADS + threadIdx.x;
      const bool in = i < n_rec;
      rk[k] = in ? c_rank[i] : 0u; cid[k] = in ? c_comm[i] : 0u; sq[k] = in ? c_seq[i] : 0u;
      if (in) todo |= 1u << k;
    }
    const u64 base_next = base + SCAT_PER_CTA;
    const bool has_next = blk + 1 < blocks_per_cta && base_next < n_rec;
    const u32 r_next = has_next ? c_rank[base_next] : 0u;     // in flight with the records
    uint4* const s_ent = s_ent_all[blk & 1][wid];
    if (e_mine.y == 0) e_mine.x = NONE;                       // an unused pair must not shadow a record of communicator 0
    s_ent[lane] = e_mine;
    __syncwarp();
#pragma unroll
    for (int k = 0; k < SCAT_PER_THREAD; ++k) {
      const u32 dr = rk[k] - r_first;
      if (dr < SCAT_LOCAL) {
        const uint4* ent = s_ent + dr * RANK_TAB_K;
        uint4 e = ent[0];
#pragma unroll
        for (int q = 1; q < RANK_TAB_K; ++q) { const uint4 x = ent[q]; if (x.x == cid[k]) e = x; }
        const u32 off = sq[k] - e.z;                          // below the first counter: wraps to a huge value
        if (e.x == cid[k] && off < e.y && ((todo >> k) & 1u)) {
          perm[e.w + off] = (u32)base + (u32)k * SCAT_THREADS + threadIdx.x;
          todo &= ~(1u << k);
        }
      }
    }
    // the next block's pairs: its first rank has arrived with this block's records
    if (has_next) e_mine = pairs_of(r_next);
    if (__any_sync(0xFFFFFFFFu, todo != 0)) {
#pragma unroll
      for (int k = 0; k < SCAT_PER_THREAD; ++k) {
        if (!((todo >> k) & 1u)) continue;
        u32 v = NONE;
        if (rk[k] < R.n_ranks) {
          const uint4 ta = R.rank_tab[(u64)rk[k] * 2], tb = R.rank_tab[(u64)rk[k] * 2 + 1];
          v = ta.x == cid[k] ? ta.y : v; v = ta.z == cid[k] ? ta.w : v;
          v = tb.x == cid[k] ? tb.y : v; v = tb.z == cid[k] ? tb.w : v;
        }
        if (v == NONE || v == RANK_TAB_OVERFLOW || cid[k] == NONE) {
          const u64 rs = resolve_slow(R, rk[k], cid[k]);
          v = (u32)rs;
          if (rs >> 32) { err |= (u32)(rs >> 32); ++rej; }
        }
        if (v == NONE) continue;
        const u32 c = v >> RANK_TAB_POS_BITS;
        const uint4 sr = srow[c];
        u64 slot;
        if (scatter_slot(R, c, sr.z, sr.w, ((u64)sr.x | ((u64)sr.y << 32)) + (u64)(v & ((1u << RANK_TAB_POS_BITS) - 1)) * sr.z, sq[k], n_slots, &slot, &err, &rej, &internal))
          perm[slot] = (u32)(base + (u64)k * SCAT_THREADS + threadIdx.x);
      }
    }
    r_first = r_next;
  }
  err = __reduce_or_sync(0xFFFFFFFFu, err);
  rej = __reduce_add_sync(0xFFFFFFFFu, rej);
  internal = __reduce_or_sync(0xFFFFFFFFu, internal);
  if ((threadIdx.x & 31) == 0) {
    if (err) atomicOr((unsigned*)&D.counters[C_ERR], err);
    count_add(D.counters, C_REJECTED, rej);
    if (internal) atomicOr((unsigned*)&D.counters[C_INTERNAL], 1u);
  }
}

}  // namespace ccld

#include "ccld_fused.cuh"
#include "ccld_large.cuh"

namespace ccld {

// ------------------------------------------------------------------------------------------------
// per-op reductions, 129 <= n <= 1024: a tile of S groups is staged in shared memory ([group][member],
// pitch n_pad + 1), reduced by one warp per group, sorted by a bitonic network over all groups at once
// ------------------------------------------------------------------------------------------------
struct MidGroup {
  u64 e_min, gbytes, med_s, mad_s, med_d, mad_d;
  u32 gfl, gop;
  u32 complete, analysed;
};

// Sort phase: full bitonic sort (merge_only = false) or only the final merge of a sequence that
// falls and then rises (merge_only = true); every group of the tile in parallel.
__device__ void mid_bitonic(u64* key, u32 S, u32 n_pad, u32 pitch, bool merge_only) {
  const u32 half = n_pad >> 1, lg_half = 31 - __clz(half);
  const u32 total = S * half;
  for (u32 k = merge_only ? n_pad : 2; k <= n_pad; k <<= 1) {
    for (u32 jj = k >> 1; jj > 0; jj >>= 1) {
      for (u32 e = threadIdx.x; e < total; e += MID_THREADS) {
        const u32 grp = e >> lg_half, q = e & (half - 1);
        const u32 i = ((q & ~(jj - 1)) << 1) | (q & (jj - 1)), l = i | jj;
        const bool up = (i & k) == 0 || k == n_pad;
        u64* a = key + grp * pitch + i; u64* b = key + grp * pitch + l;
        const u64 va = *a, vb = *b;
        if ((va > vb) == up) { *a = vb; *b = va; }
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(MID_THREADS) k_reduce_mid(const WinDesc* __restrict__ wd, const Tile* __restrict__ tiles,
                                                            TileSum* __restrict__ sums, Registry R, Params P, i64 now) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const Tile t = tiles[blockIdx.x];
  const WinDesc& D = wd[t.w];
  const u32 c = t.c, n = R.comm_n[c];
  const RangeRow row = D.ranges[c];
  const u32* mem = R.members + R.comm_moff[c];
  const u32 n_pad = mid_npad(n), pitch = n_pad + 1, S = t.count, S_max = MID_ELEMS / n_pad;
  const u32 cap = S_max * pitch;
  // shared-memory carve-up
  u64* s_te = (u64*)smem_raw;            // enter time
  u64* s_du = s_te + cap;                // duration
  u64* s_key = s_du + cap;               // sort buffer
  u64* s_by = s_key + cap;               // bytes
  u32* s_idx = (u32*)(s_by + cap);       // record index
  u32* s_ch = s_idx + cap;               // max(send_chg, recv_chg)
  u8* s_op = (u8*)(s_ch + cap);
  u8* s_st = s_op + cap;                 // 1 present, 2 in flight, 4 bad time
  MidGroup* s_g = (MidGroup*)(((uintptr_t)(s_st + cap) + 15) & ~(uintptr_t)15);
  __shared__ u32 s_cnt[8];
  __shared__ u64 s_brng[MID_THREADS / 32];
  __shared__ u32 s_bk[MID_THREADS / 32], s_rounds[MID_THREADS / 32];
  u64 w_brng = 0; u32 w_bk = NONE, w_rounds = 0;          // this warp's Eq. 2 candidate and round count (lane 0)

  const u64 slot_t = row.slot0 + (u64)t.seq_off * n;      // first slot of the tile
  const u64 g_t = row.group0 + t.seq_off;                  // first group of the tile
  const u32 n_el = S * n;
  if (threadIdx.x < 8) s_cnt[threadIdx.x] = 0;
  // 1. record indices, coalesced along the slot order
  for (u32 p = threadIdx.x >> 5; p < n; p += MID_THREADS / 32) {
    const u32* __restrict__ pm = D.perm + perm_at(row, t.seq_off, p);
    for (u32 jg = threadIdx.x & 31; jg < S; jg += 32) s_idx[jg * pitch + p] = pm[jg];
  }
  __syncthreads();
  // 2. gather: consecutive threads walk consecutive op counters of one member
  for (u32 e = threadIdx.x; e < n_el; e += MID_THREADS) {
    const u32 p = e / S, jg = e - p * S, a = jg * pitch + p;
    const u32 idx = s_idx[a];
    u64 te = 0, du = 0, by = 0; u32 ch = 0; u8 op = 0, st = 0;
    if (idx != NONE) {
      const i64 x = D.t_enter[idx], y = D.t_exit[idx];
      by = D.bytes[idx]; op = D.op[idx];
      if (D.send_chg != nullptr) { const u32 sc = D.send_chg[idx], rc = D.recv_chg[idx]; ch = sc > rc ? sc : rc; }
      st = 1 | (y == -1 ? 2 : ((x < 0 || y < x) ? 4 : 0));
      te = (u64)x; du = (u64)(y - x);
    }
    s_te[a] = te; s_du[a] = du; s_by[a] = by; s_ch[a] = ch; s_op[a] = op; s_st[a] = st;
  }
  __syncthreads();
  // 3. one warp per group: cross-rank reductions
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u32 c_comp = 0, c_inc = 0, c_bar = 0, c_an = 0, c_mis = 0, c_pres = 0;
  for (u32 jg = wid; jg < S; jg += MID_THREADS / 32) {
    const u32 b = jg * pitch;
    u32 npres = 0, first = NONE, stor = 0;
    for (u32 p = lane; p < n; p += 32) { const u32 st = s_st[b + p]; if (st & 1) { ++npres; first = first == NONE ? p : first; } stor |= st; }
    npres = __reduce_add_sync(0xFFFFFFFFu, npres); first = __reduce_min_sync(0xFFFFFFFFu, first); stor = __reduce_or_sync(0xFFFFFFFFu, stor);
    const bool have_first = first != NONE;
    const u64 gbytes = have_first ? s_by[b + first] : 0; const u32 gop = have_first ? s_op[b + first] : 0;
    const bool inflight = stor & 2, bad_time = stor & 4, complete = npres == n && !inflight && !bad_time;
    const bool barrier = have_first && gop == CCLD_OP_ALLREDUCE && gbytes < P.barrier_bytes;
    u32 mism = 0; i64 age = -1;
    u64 e_min = U64_MAX_, tmax = 0, tmin = U64_MAX_; i64 x_max = INT64_MIN; u32 pmax = NONE, pmin = NONE; u64 chk = 0;
    for (u32 p = lane; p < n; p += 32) {
      const u32 st = s_st[b + p];
      if (!(st & 1)) continue;
      if (s_op[b + p] != gop || s_by[b + p] != gbytes) mism = 1;
      const u64 te = s_te[b + p], du = s_du[b + p];
      if (st & 2) { const i64 ag = now - (i64)te; age = ag > age ? ag : age; }
      e_min = te < e_min ? te : e_min;
      const i64 tx = (i64)(te + du); x_max = tx > x_max ? tx : x_max;
      if (pmax == NONE || du > tmax) { tmax = du; pmax = p; }
      if (pmin == NONE || du < tmin) { tmin = du; pmin = p; }
      const u64 ck = ((u64)s_ch[b + p] << 32) | (u64)(NONE - p);        // most changes, then lowest position
      chk = ck > chk ? ck : chk;
    }
    mism = __reduce_or_sync(0xFFFFFFFFu, mism);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const i64 ag = (i64)shfl_xor64((u64)age, d); age = ag > age ? ag : age;
      const u64 em = shfl_xor64(e_min, d); e_min = em < e_min ? em : e_min;
      const i64 xm = (i64)shfl_xor64((u64)x_max, d); x_max = xm > x_max ? xm : x_max;
      const u64 ck = shfl_xor64(chk, d); chk = ck > chk ? ck : chk;
      const u64 tM = shfl_xor64(tmax, d); const u32 pM = __shfl_xor_sync(0xFFFFFFFFu, pmax, d);
      if (pM != NONE && (pmax == NONE || tM > tmax || (tM == tmax && pM < pmax))) { tmax = tM; pmax = pM; }
      const u64 tm = shfl_xor64(tmin, d); const u32 pm = __shfl_xor_sync(0xFFFFFFFFu, pmin, d);
      if (pm != NONE && (pmin == NONE || tm < tmin || (tm == tmin && pm < pmin))) { tmin = tm; pmin = pm; }
    }
    u32 gfl = (mism ? CCLD_G_OPSET_MISMATCH : 0) | (barrier ? CCLD_G_BARRIER : 0) | (inflight ? CCLD_G_INFLIGHT : 0) |
              (bad_time ? CCLD_G_BAD_TIME : 0) | (complete ? CCLD_G_COMPLETE : CCLD_G_INCOMPLETE);
    const bool analysed = complete && !barrier && n >= P.min_group;
    if (analysed) gfl |= CCLD_G_ANALYSED;
    const bool hang = !complete && inflight && age > P.hang_ns && !barrier;
    if (hang) gfl |= CCLD_G_HANG_ALERT;
    if (lane == 0) {
      const u64 g = g_t + jg, G = D.n_groups;
      if (hang) raise_alert(D, R.comm_id[c], row.seq_lo + t.seq_off + jg, age);
      MidGroup mg; mg.e_min = e_min; mg.gbytes = gbytes; mg.gop = gop; mg.gfl = gfl; mg.complete = complete; mg.analysed = analysed;
      mg.med_s = mg.mad_s = mg.med_d = mg.mad_d = 0;
      s_g[jg] = mg;
      i64 span = 0; double gb = 0.0;
      if (complete) {
        span = x_max - (i64)e_min;
        double num, den; bus_factor(gop, n, &num, &den);
        gb = busbw((double)gbytes * num, den, span);
      }
      D.gi64[(u64)GI_E_MIN * G + g] = complete ? (i64)e_min : 0;
      D.gi64[(u64)GI_T_MAX * G + g] = complete ? (i64)tmax : 0; D.gi64[(u64)GI_T_MIN * G + g] = complete ? (i64)tmin : 0;
      D.gi64[(u64)GI_SPAN * G + g] = span;
      D.gu32[(u64)GU_RANK_TMIN * G + g] = complete ? mem[pmin] : 0; D.gu32[(u64)GU_RANK_TMAX * G + g] = complete ? mem[pmax] : 0;
      D.gu32[(u64)GU_MAX_CHG * G + g] = complete ? (u32)(chk >> 32) : 0;
      D.gu32[(u64)GU_RANK_MAX_CHG * G + g] = complete ? mem[NONE - (u32)chk] : 0;
      D.gu32[(u64)GU_N_PRESENT * G + g] = npres; D.gu32[(u64)GU_GFLAGS * G + g] = gfl;
      D.gbw[g] = gb;
      c_comp += complete; c_inc += !complete; c_bar += barrier; c_an += analysed; c_mis += mism; c_pres += npres;
      if (complete && !barrier) { ++w_rounds; best_merge(w_brng, w_bk, tmax - tmin, t.seq_off + jg); }
    }
  }
  if (lane == 0) { s_brng[wid] = w_brng; s_bk[wid] = w_bk; s_rounds[wid] = w_rounds; }
  __syncthreads();
  const u32 k_med = (n - 1) >> 1;
  // 4. arrival skew: sort, median, deviations, merge, MAD
  for (u32 e = threadIdx.x; e < S * n_pad; e += MID_THREADS) {
    const u32 jg = e / n_pad, i = e - jg * n_pad;
    s_key[jg * pitch + i] = (i < n && s_g[jg].analysed) ? s_te[jg * pitch + i] - s_g[jg].e_min : U64_MAX_;
  }
  __syncthreads();
  mid_bitonic(s_key, S, n_pad, pitch, false);
  for (u32 jg = threadIdx.x; jg < S; jg += MID_THREADS) s_g[jg].med_s = s_key[jg * pitch + k_med];
  __syncthreads();
  for (u32 e = threadIdx.x; e < S * n_pad; e += MID_THREADS) {
    const u32 jg = e / n_pad, i = e - jg * n_pad;
    if (i < n) s_key[jg * pitch + i] = absdiff(s_key[jg * pitch + i], s_g[jg].med_s);
  }
  __syncthreads();
  mid_bitonic(s_key, S, n_pad, pitch, true);
  for (u32 jg = threadIdx.x; jg < S; jg += MID_THREADS) {
    s_g[jg].mad_s = s_key[jg * pitch + k_med];
    const u64 g = g_t + jg, G = D.n_groups; const bool an = s_g[jg].analysed;
    D.gi64[(u64)GI_MED_SKEW * G + g] = an ? (i64)s_g[jg].med_s : 0; D.gi64[(u64)GI_MAD_SKEW * G + g] = an ? (i64)s_g[jg].mad_s : 0;
  }
  __syncthreads();
  // 5. duration: the same
  for (u32 e = threadIdx.x; e < S * n_pad; e += MID_THREADS) {
    const u32 jg = e / n_pad, i = e - jg * n_pad;
    s_key[jg * pitch + i] = (i < n && s_g[jg].analysed) ? s_du[jg * pitch + i] : U64_MAX_;
  }
  __syncthreads();
  mid_bitonic(s_key, S, n_pad, pitch, false);
  for (u32 jg = threadIdx.x; jg < S; jg += MID_THREADS) s_g[jg].med_d = s_key[jg * pitch + k_med];
  __syncthreads();
  for (u32 e = threadIdx.x; e < S * n_pad; e += MID_THREADS) {
    const u32 jg = e / n_pad, i = e - jg * n_pad;
    if (i < n) s_key[jg * pitch + i] = absdiff(s_key[jg * pitch + i], s_g[jg].med_d);
  }
  __syncthreads();
  mid_bitonic(s_key, S, n_pad, pitch, true);
  for (u32 jg = threadIdx.x; jg < S; jg += MID_THREADS) {
    s_g[jg].mad_d = s_key[jg * pitch + k_med];
    const u64 g = g_t + jg, G = D.n_groups; const bool an = s_g[jg].analysed;
    D.gi64[(u64)GI_MED_DUR * G + g] = an ? (i64)s_g[jg].med_d : 0; D.gi64[(u64)GI_MAD_DUR * G + g] = an ? (i64)s_g[jg].mad_d : 0;
  }
  __syncthreads();
  // 6. flags and votes, in slot order (coalesced byte stores)
  u32 n_fs = 0, n_fd = 0;
  for (u32 e = threadIdx.x; e < n_el; e += MID_THREADS) {
    const u32 jg = e / n, p = e - jg * n, a = jg * pitch + p;
    const MidGroup& mg = s_g[jg];
    u8 f = CCLD_F_NOT_ANALYSED;
    if (!(s_st[a] & 1)) f |= CCLD_F_MISSING;
    else if (mg.analysed) {
      const u64 sk = s_te[a] - mg.e_min, du = s_du[a];
      const bool so = mul_gt(absdiff(sk, mg.med_s), 1000u, mg.mad_s, P.k_milli), sh = sk > mg.med_s;
      const bool dq = mul_gt(absdiff(du, mg.med_d), 1000u, mg.mad_d, P.k_milli), dh = du > mg.med_d;
      f = (so ? CCLD_F_SKEW_OUT : 0) | (dq ? CCLD_F_DUR_OUT : 0) | (sh ? CCLD_F_SKEW_HI : 0) | (dh ? CCLD_F_DUR_HI : 0);
      if (so) { ++n_fs; atomicAdd(&R.votes[(u64)mem[p] * 4 + (sh ? 0 : 1)], 1u); }
      if (dq) { ++n_fd; atomicAdd(&R.votes[(u64)mem[p] * 4 + (dh ? 2 : 3)], 1u); }
    }
    D.flags[slot_t + e] = f;
  }
  // arrival skew = largest enter time minus the smallest, one warp per group
  for (u32 jg = wid; jg < S; jg += MID_THREADS / 32) {
    u64 mx = 0;
    if (s_g[jg].complete) {
      for (u32 p = lane; p < n; p += 32) { const u64 v = s_te[jg * pitch + p]; mx = v > mx ? v : mx; }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) { const u64 o = shfl_xor64(mx, d); mx = o > mx ? o : mx; }
    }
    if (lane == 0) D.gi64[(u64)GI_ARRIVAL_SKEW * D.n_groups + g_t + jg] = s_g[jg].complete ? (i64)(mx - s_g[jg].e_min) : 0;
  }
  // 7. per-rank bus bandwidth: thread p sums member p over the tile's groups
  u32 n_bwc = 0;
  for (u32 jg = 0; jg < S; ++jg) n_bwc += (s_g[jg].complete && !(s_g[jg].gfl & CCLD_G_BARRIER)) ? 1u : 0u;
  if (n_bwc) {
    for (u32 p = threadIdx.x; p < n; p += MID_THREADS) {
      double v = 0.0;
      for (u32 jg = 0; jg < S; ++jg) {
        const MidGroup& mg = s_g[jg];
        if (!mg.complete || (mg.gfl & CCLD_G_BARRIER)) continue;
        double num, den; bus_factor(mg.gop, n, &num, &den);
        v += busbw((double)mg.gbytes * num, den, (i64)s_du[jg * pitch + p]);
      }
      atomicAdd(&R.bw_sum[mem[p]], v);
      atomicAdd(&R.bw_cnt[mem[p]], n_bwc);
    }
  }
  // 8. counters
  n_fs = __reduce_add_sync(0xFFFFFFFFu, n_fs); n_fd = __reduce_add_sync(0xFFFFFFFFu, n_fd);
  if (lane == 0) {
    atomicAdd(&s_cnt[0], c_comp); atomicAdd(&s_cnt[1], c_inc); atomicAdd(&s_cnt[2], c_bar); atomicAdd(&s_cnt[3], c_an);
    atomicAdd(&s_cnt[4], c_mis); atomicAdd(&s_cnt[5], c_pres); atomicAdd(&s_cnt[6], n_fs); atomicAdd(&s_cnt[7], n_fd);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 brng = s_brng[0]; u32 bk = s_bk[0], rounds = s_rounds[0];
    for (int q = 1; q < MID_THREADS / 32; ++q) { best_merge(brng, bk, s_brng[q], s_bk[q]); rounds += s_rounds[q]; }
    TileSum ts; ts.best_rng = brng; ts.best_k = bk; ts.n_rounds = rounds; ts.n_an = s_cnt[3]; ts.pad = 0;
    sums[blockIdx.x] = ts;
    count_add(D.counters, C_COMPLETE, s_cnt[0]); count_add(D.counters, C_INCOMPLETE, s_cnt[1]); count_add(D.counters, C_BARRIER, s_cnt[2]);
    count_add(D.counters, C_ANALYSED, s_cnt[3]); count_add(D.counters, C_MISMATCH, s_cnt[4]); count_add(D.counters, C_PRESENT, s_cnt[5]);
    count_add(D.counters, C_FLAG_SKEW, s_cnt[6]); count_add(D.counters, C_FLAG_DUR, s_cnt[7]);
  }
}

inline size_t mid_smem_bytes(u32 n_pad_min) {
  // cap = (MID_ELEMS / n_pad) * (n_pad + 1) is largest for the smallest n_pad
  size_t cap = (size_t)(MID_ELEMS / n_pad_min) * (n_pad_min + 1);
  return cap * (4 * 8 + 2 * 4 + 2) + 16 + (MID_ELEMS / n_pad_min) * sizeof(MidGroup);
}

// ------------------------------------------------------------------------------------------------
// window decision per communicator (Sec. 4.2.1 Eq. 1-3, Sec. 4.2.2 Eq. 4): one warp per
// communicator walks the windows of the batch in order
// ------------------------------------------------------------------------------------------------
// Stage 1, one warp per (communicator, window), all windows at once: everything of the window decision that does not
// depend on the state carried from window to window - the round and analysed-op counts, the round Eq. 2 selects with its
// T_max / T_min and the ranks the location step would name - goes into the communicator's verdict row.
__global__ void __launch_bounds__(128) k_window_rounds(const WinDesc* __restrict__ wd, Registry R) {
  const u32 c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (c >= R.n_comms) return;
  const WinDesc& D = wd[blockIdx.y];
  const RangeRow row = D.ranges[c];
  if (row.n_seq == 0) return;
  const u32 n = R.comm_n[c], cls = comm_class(n);
  const u32* mem = R.members + R.comm_moff[c];
  const u64 G = D.n_groups;
  const i64* t_max = D.gi64 + (u64)GI_T_MAX * G + row.group0;
  const i64* t_min = D.gi64 + (u64)GI_T_MIN * G + row.group0;
  // round counts and the Eq. 2 candidate come from the tile summaries the reduce kernels left behind
  const TileSum* ts = D.tsum[cls <= 1 ? 0 : cls - 1] + row.tile0;
  const u32 nt = row.n_units;
  u32 n_rounds = 0, n_an = 0;
  u64 best_rng = 0; u32 best_k = NONE;
  bool redo = false;                                     // a unit left groups to the deferred kernel: its summary is partial
  for (u32 q = lane; q < nt; q += 32) {
    const TileSum x = ts[q];
    n_rounds += x.n_rounds; n_an += x.n_an;
    best_merge(best_rng, best_k, x.best_rng, x.best_k);
    redo = redo || x.pad != 0;
  }
  if (__any_sync(0xFFFFFFFFu, redo)) {
    // recount the communicator's window from the per-op rows
    const u32* gfl = D.gu32 + (u64)GU_GFLAGS * G + row.group0;
    n_rounds = 0; n_an = 0; best_rng = 0; best_k = NONE;
    for (u32 k = lane; k < row.n_seq; k += 32) {
      const u32 f = gfl[k];
      if ((f & CCLD_G_COMPLETE) && !(f & CCLD_G_BARRIER)) { ++n_rounds; best_merge(best_rng, best_k, (u64)(t_max[k] - t_min[k]), k); }
      if (f & CCLD_G_ANALYSED) ++n_an;
    }
  }
  n_rounds = __reduce_add_sync(0xFFFFFFFFu, n_rounds); n_an = __reduce_add_sync(0xFFFFFFFFu, n_an);
  best_warp_reduce(best_rng, best_k);
  // analysed ops of this window count towards every member's denominator
  if (n_an) for (u32 p = lane; p < n; p += 32) atomicAdd(&R.ops[mem[p]], n_an);
  if (lane == 0) {
    ccld_comm_verdict v;
    v.comm = R.comm_id[c]; v.n_rounds = n_rounds; v.sel_seq = NONE; v.cls = 0; v.slow_detected = 0; v.located = 0;
    v.baseline_static = 0; v.rate_source = 0; v.root_comp = NONE; v.root_comm = NONE;
    v.t_max = 0; v.t_min = 0; v.R = 0.0; v.P = 0.0; v.t_base = 0; v.rounds_total = 0; v.m = 0; v.slow_count = 0;
    if (best_k != NONE) {
      v.sel_seq = row.seq_lo + best_k; v.t_max = t_max[best_k]; v.t_min = t_min[best_k];
      const u64 gq = row.group0 + best_k;
      v.root_comp = D.gu32[(u64)GU_RANK_TMIN * G + gq];
      const u32 mc = D.gu32[(u64)GU_MAX_CHG * G + gq];
      if (mc > 0) { v.root_comm = D.gu32[(u64)GU_RANK_MAX_CHG * G + gq]; v.rate_source = 0; }
      else { v.root_comm = D.gu32[(u64)GU_RANK_TMAX * G + gq]; v.rate_source = 1; }
    }
    D.comm_rows[row.row_idx] = v;
  }
}

// Stage 2, one warp per communicator, windows in order: the recurrences - Eq. 1's baseline, which reads the per-op rows
// until m is fixed, and the repetition counter - and with them Eq. 3, Eq. 4 and the location rule, which complete the
// row stage 1 wrote. What a window needs is fetched ahead (range rows two windows, the stage-1 row and the result
// pointers one window), so the walk waits for arithmetic only.
__global__ void __launch_bounds__(128) k_window_decide(const WinDesc* __restrict__ wd, u32 nw, Registry R, Params P) {
  const u32 c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (c >= R.n_comms) return;
  CommState st = R.state[c];
  struct Res { const RangeRow* ranges; u64 n_groups; const i64* gi64; const u32* gu32; ccld_comm_verdict* comm_rows; };   // pointers of a window
  struct Part { u32 n_rounds, sel_seq, root_comp, root_comm, rate_source; i64 t_max, t_min; };    // what stage 1 left in the row
  // three steps, each on values fetched during an earlier window: descriptor -> range row -> stage-1 row
  auto load_res = [&](u32 w) {
    Res r = {nullptr, 0, nullptr, nullptr, nullptr};
    if (w < nw) { r.ranges = wd[w].ranges; r.n_groups = wd[w].n_groups; r.gi64 = wd[w].gi64; r.gu32 = wd[w].gu32; r.comm_rows = wd[w].comm_rows; }
    return r;
  };
  auto load_row = [&](const Res& r) { RangeRow x = {0, 0, 0, 0, 0, 0, 0, 0}; if (r.ranges != nullptr) x = r.ranges[c]; return x; };
  auto load_part = [&](const Res& r, const RangeRow& row) {
    Part x = {0, NONE, NONE, NONE, 0, 0, 0};
    if (r.comm_rows != nullptr && row.n_seq != 0) {
      const ccld_comm_verdict* v = r.comm_rows + row.row_idx;
      x.n_rounds = v->n_rounds; x.sel_seq = v->sel_seq; x.root_comp = v->root_comp; x.root_comm = v->root_comm;
      x.rate_source = v->rate_source; x.t_max = v->t_max; x.t_min = v->t_min;
    }
    return x;
  };
  Res res_a = load_res(0), res_b = load_res(1), res_c = load_res(2);
  RangeRow row_a = load_row(res_a), row_b = load_row(res_b);
  Part part_a = load_part(res_a, row_a);
  for (u32 w = 0; w < nw; ++w) {
    const RangeRow row = row_a; const Res D = res_a; const Part pt = part_a;
    part_a = load_part(res_b, row_b);                    // window w + 1
    row_a = row_b; row_b = load_row(res_c);              // window w + 2
    res_a = res_b; res_b = res_c; res_c = load_res(w + 3);
    if (row.n_seq == 0) continue;
    const u64 G = D.n_groups;
    const u32 n_rounds = pt.n_rounds;
    // Eq. 1: rounds feed the baseline, in op-counter order, until m is fixed
    u32 walked = 0;
    if (st.m == 0 && n_rounds > 0) {
      const u32* gfl = D.gu32 + (u64)GU_GFLAGS * G + row.group0;
      const i64* e_min = D.gi64 + (u64)GI_E_MIN * G + row.group0;
      const i64* t_max = D.gi64 + (u64)GI_T_MAX * G + row.group0;
      for (u32 k0 = 0; k0 < row.n_seq && st.m == 0; k0 += 32) {
        const u32 k = k0 + lane;
        const u32 f = k < row.n_seq ? gfl[k] : 0;
        const bool round = (f & CCLD_G_COMPLETE) && !(f & CCLD_G_BARRIER);
        u32 rem = __ballot_sync(0xFFFFFFFFu, round);
        i64 em = 0, tM = 0;
        if (round) { em = e_min[k]; tM = t_max[k]; }
        while (rem && st.m == 0) {
          const int src = __ffs(rem) - 1; rem &= rem - 1;
          const i64 em_s = __shfl_sync(0xFFFFFFFFu, em, src), tM_s = __shfl_sync(0xFFFFFFFFu, tM, src);
          if (st.rounds == 0) st.t_first = em_s;
          if (st.rounds == (u64)P.m_max_rounds || (st.rounds > 0 && em_s - st.t_first >= P.m_max_ns)) st.m = st.rounds;
          else st.sum_m += tM_s;
          ++st.rounds; ++walked;
        }
      }
    }
    st.rounds += n_rounds - walked;
    if (lane == 0) {
      ccld_comm_verdict v;
      v.comm = R.comm_id[c]; v.n_rounds = n_rounds; v.sel_seq = pt.sel_seq; v.cls = 0; v.slow_detected = 0; v.located = 0;
      v.baseline_static = st.m == 0; v.rate_source = 0; v.root_comp = NONE; v.root_comm = NONE;
      v.t_max = pt.t_max; v.t_min = pt.t_min; v.R = 0.0; v.P = 0.0;
      v.t_base = st.m > 0 ? st.sum_m / (i64)st.m : P.tbase_init_ns;
      v.rounds_total = st.rounds; v.m = st.m;
      if (pt.sel_seq != NONE) {
        v.R = (double)(v.t_max - v.t_base) / (double)v.t_base;                                     // Eq. 3
        const bool slow = v.t_max > v.t_base && mul_gt((u64)(v.t_max - v.t_base), 1000u, (u64)v.t_base, P.theta_slow_milli);
        v.slow_detected = slow;
        if (slow) {
          ++st.slow_count;
          v.located = st.slow_count > (u64)P.slow_rep_threshold;
          const u64 num = (u64)(v.t_max - v.t_min), den = (u64)(v.t_max - v.t_base);
          v.P = (double)num / (double)den;                                                         // Eq. 4
          v.cls = mul_gt(num, 1000u, den, P.beta_milli) ? 1u : (mul_lt(num, 1000u, den, P.alpha_milli) ? 2u : 3u);
          v.root_comp = pt.root_comp; v.root_comm = pt.root_comm; v.rate_source = pt.rate_source;
        }
      }
      v.slow_count = st.slow_count;
      D.comm_rows[row.row_idx] = v;
    }
    st.slow_count = __shfl_sync(0xFFFFFFFFu, st.slow_count, 0);
  }
  if (lane == 0) R.state[c] = st;
}

// ------------------------------------------------------------------------------------------------
// hang location (Sec. 4.2.2, Fig. 6): one CTA
// ------------------------------------------------------------------------------------------------
struct HangArgs {
  u32 c, seq, n_frames, n_channels;
  const u32 *f_rank, *f_comm, *f_seq, *progress;
  u8* entered; u8* done;     // [n] scratch
  u32* frame;                // [n] scratch
  u64* tot;                  // [n] scratch
  u32* roots; u32 roots_cap; // device list
  ccld_hang_verdict* out;    // device copy of the struct (pointer fields unused)
  const u32* head;           // [n] tree communicators: lowest position of each member's layer; null for a ring
};

__device__ __forceinline__ void hang_locate_cta(const WinDesc& D, const Registry& R, const HangArgs& A) {
  __shared__ u64 s_red64[32];
  __shared__ u32 s_red32[32];
  __shared__ u32 s_base;
  const u32 c = A.c, n = R.comm_n[c], cid = R.comm_id[c];
  const u32* mem = R.members + R.comm_moff[c];
  const RangeRow row = D.ranges[c];
  for (u32 p = threadIdx.x; p < n; p += blockDim.x) { A.entered[p] = 0; A.done[p] = 0; A.frame[p] = NONE; A.tot[p] = 0; }
  __syncthreads();
  // a member has entered if it reported this or a later op counter
  if (row.n_seq > 0 && A.seq <= row.seq_lo + (row.n_seq - 1)) {
    const u32 s_first = A.seq > row.seq_lo ? A.seq - row.seq_lo : 0;
    const u64 cnt = (u64)(row.n_seq - s_first) * n;
    for (u64 e = threadIdx.x; e < cnt; e += blockDim.x) {
      const u32 so = s_first + (u32)(e / n), p = (u32)(e % n);
      const u32 idx = D.perm[perm_at(row, so, p)];
      if (idx != NONE) {
        A.entered[p] = 1;
        if (row.seq_lo + so == A.seq && D.t_exit[idx] != -1) A.done[p] = 1;
      }
    }
  }
  // progress frames of this op: the first frame uploaded for a member counts
  for (u32 f = threadIdx.x; f < A.n_frames; f += blockDim.x) {
    if (A.f_comm[f] != cid || A.f_seq[f] != A.seq) continue;
    const u32 p = pos_lookup(R, A.f_rank[f], c);
    if (p != NONE) atomicMin(&A.frame[p], f);
  }
  __syncthreads();
  u32 n_ne = 0, n_ok = 0, n_missing = 0; u64 mn = U64_MAX_;
  for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
    n_ne += !A.entered[p]; n_ok += A.done[p];
    const u32 f = A.frame[p];
    u64 tot = 0;
    if (f == NONE) ++n_missing;
    else for (u32 ch = 0; ch < A.n_channels; ++ch) tot += (u64)A.progress[((u64)f * A.n_channels + ch) * 2] + A.progress[((u64)f * A.n_channels + ch) * 2 + 1];
    A.tot[p] = tot; mn = tot < mn ? tot : mn;
  }
  n_ne = block_reduce(n_ne, OpAddU32(), s_red32);
  n_ok = block_reduce(n_ok, OpAddU32(), s_red32);
  n_missing = block_reduce(n_missing, OpAddU32(), s_red32);
  mn = block_reduce(mn, OpMinU64(), s_red64);
  __syncthreads();
  const u32 cls = n_ne > 0 ? 1u : (n_ok > 0 ? 2u : 3u);
  u32 n_roots = 0, stuck = 0; u64 min_total = 0;
  if (cls == 3 && A.head != nullptr) {
    // tree (Sec. 4.2.1): counters are comparable inside a layer only. The lowest position of a layer walks the layer:
    // its minimum, the first member that holds it, its maximum. The layer whose minimum is furthest behind its maximum
    // names the root; equal gaps: the lowest position; no gap anywhere: nobody.
    u64 lag = 0; u32 cand = NONE;
    for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
      if (A.head[p] != p) continue;
      u64 lmn = A.tot[p], lmx = lmn; u32 at = p;
      for (u32 x = p + 1; x < n; ++x) {
        if (A.head[x] != p) continue;
        const u64 t = A.tot[x];
        if (t < lmn) { lmn = t; at = x; }
        lmx = t > lmx ? t : lmx;
      }
      const u64 g = lmx - lmn;
      if (g > lag || (g == lag && g > 0 && at < cand)) { lag = g; cand = at; }
    }
    const u64 best = block_reduce(lag, OpMaxU64(), s_red64);
    if (lag != best || best == 0) cand = NONE;
    const u32 root = block_reduce(cand, OpMinU32(), s_red32);
    if (root != NONE) {
      n_roots = 1; min_total = A.tot[root];
      if (threadIdx.x == 0) {
        if (A.roots_cap > 0) A.roots[0] = mem[root];
        const u32 f = A.frame[root];
        if (f != NONE && A.n_channels > 0) {
          u32 s = NONE;
          for (u32 ch = 0; ch < A.n_channels; ++ch) { const u32 r = A.progress[((u64)f * A.n_channels + ch) * 2 + 1]; s = r < s ? r : s; }
          stuck = s;
        }
      }
    }
  } else if (cls == 3) {
    // fewest counters; among equals the most upstream of a run (predecessor ahead), then the lowest position
    u32 up = NONE, any = NONE;
    for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
      if (A.tot[p] != mn) continue;
      any = p < any ? p : any;
      if (A.tot[(p + n - 1) % n] > mn) up = p < up ? p : up;
    }
    up = block_reduce(up, OpMinU32(), s_red32);
    any = block_reduce(any, OpMinU32(), s_red32);
    const u32 root = up != NONE ? up : any;
    n_roots = 1; min_total = mn;
    if (threadIdx.x == 0) {
      if (A.roots_cap > 0) A.roots[0] = mem[root];
      const u32 f = A.frame[root];
      if (f != NONE && A.n_channels > 0) {
        u32 s = NONE;
        for (u32 ch = 0; ch < A.n_channels; ++ch) { const u32 r = A.progress[((u64)f * A.n_channels + ch) * 2 + 1]; s = r < s ? r : s; }
        stuck = s;
      }
    }
  } else {
    // ordered compaction of the not-entered (H1) or not-hung (H2) members
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (u32 p0 = 0; p0 < n; p0 += blockDim.x) {
      const u32 p = p0 + threadIdx.x;
      const bool sel = p < n && (cls == 1 ? !A.entered[p] : A.done[p] != 0);
      const u32 bal = __ballot_sync(0xFFFFFFFFu, sel);
      const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
      __syncthreads();
      if (lane == 0) s_red32[wid] = __popc(bal);
      __syncthreads();
      u32 off = s_base;
      for (u32 q = 0; q < wid; ++q) off += s_red32[q];
      off += __popc(bal & ((1u << lane) - 1));
      if (sel && off < A.roots_cap) A.roots[off] = mem[p];
      __syncthreads();
      if (threadIdx.x == 0) { u32 tot = 0; for (u32 q = 0; q < blockDim.x / 32; ++q) tot += s_red32[q]; s_base += tot; }
      __syncthreads();
    }
    n_roots = s_base;
  }
  if (threadIdx.x == 0) {
    ccld_hang_verdict v;
    v.cls = cls; v.n_roots_total = n_roots; v.n_not_entered = n_ne; v.n_hung = n - n_ok; v.n_not_hung = n_ok;
    v.n_missing_frames = cls == 3 ? n_missing : 0; v.stuck_step = stuck; v.n_members = n; v.min_total = min_total;
    v.roots = nullptr; v.roots_cap = 0;
    *A.out = v;
  }
}

__global__ void __launch_bounds__(1024) k_hang_locate(const WinDesc* __restrict__ wd, Registry R, HangArgs A) { hang_locate_cta(wd[0], R, A); }

// every alert of a window in one launch: one CTA per alert, each with its own scratch and output
__global__ void __launch_bounds__(1024) k_hang_locate_many(const WinDesc* __restrict__ wd, Registry R, const HangArgs* __restrict__ args) {
  const HangArgs A = args[blockIdx.x];
  hang_locate_cta(wd[0], R, A);
}

}  // namespace ccld
#include "ccld_tree.cuh"
namespace ccld {

// ------------------------------------------------------------------------------------------------
// suspects and ordered lists
// ------------------------------------------------------------------------------------------------
__global__ void k_suspects(Registry R, Params P, ccld_suspect* __restrict__ out, u32 cap, u32* __restrict__ count) {
  const u32 r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R.n_ranks) return;
  const u32 ops = R.ops[r];
  if (ops == 0) return;
  const u32 cnt = R.bw_cnt[r];
  const double bw = cnt ? R.bw_sum[r] / (double)cnt : 0.0;
  const u32 v[2] = {R.votes[(u64)r * 4 + 0], R.votes[(u64)r * 4 + 2]};
  for (u32 kind = 1; kind <= 2; ++kind) {
    if ((u64)v[kind - 1] * 1000u >= (u64)P.vote_rep_milli * ops) {
      const u32 k = atomicAdd(count, 1u);
      if (k < cap) { ccld_suspect s; s.kind = kind; s.rank = r; s.votes = v[kind - 1]; s.ops = ops; s.mean_busbw = bw; out[k] = s; }
    }
  }
}

// Rank-by-counting sort of short lists: element i goes to the number of elements that precede it.
__global__ void k_rank_sort_suspects(const ccld_suspect* __restrict__ in, u32 n, ccld_suspect* __restrict__ out) {
  const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const ccld_suspect a = in[i];
  u32 before = 0;
  for (u32 j = 0; j < n; ++j) {
    const ccld_suspect b = in[j];
    const bool lt = b.kind != a.kind ? b.kind < a.kind : (b.votes != a.votes ? b.votes > a.votes : b.rank < a.rank);
    before += lt;
  }
  out[before] = a;
}

__global__ void k_rank_sort_alerts(const ccld_hang_alert* __restrict__ in, u32 n, ccld_hang_alert* __restrict__ out, Registry R) {
  const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const ccld_hang_alert a = in[i];
  const u32 ca = comm_lookup(R, a.comm);
  u32 before = 0;
  for (u32 j = 0; j < n; ++j) {
    const ccld_hang_alert b = in[j];
    const u32 cb = comm_lookup(R, b.comm);
    before += cb != ca ? cb < ca : b.seq < a.seq;
  }
  out[before] = a;
}

}  // namespace ccld
