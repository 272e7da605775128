// Per-op reductions, median / MAD, flags and votes for communicators of more than 1,024 ranks (sm_100a).
//
// A group of thousands of members has its records spread over as many places of the upload, and its order statistics
// need every key several times. The work is therefore cut in two:
//
//   k_large_stage            one pass over the records of a tile (LARGE_SEQS consecutive op counters of one communicator,
//                            LS_MEMBERS members per CTA). Lanes run along the op counter first: the eight record indices
//                            of a member are one 32-byte sector of the member-major permutation, and in a rank-major
//                            upload the eight records are neighbours too, so every gather of a warp fetches whole
//                            sectors. Times become 32-bit keys (enter-time offset from the group's first member, duration)
//                            and leave, transposed through shared memory, as two contiguous arrays per group; the extrema,
//                            the op-set check and the rate column are reduced on the way and merged per group with atomics.
//   k_reduce_large           the order statistics. A CTA works on G groups of a tile side by side (G = 8, 4, 2 or 1: a
//                            thread keeps its share of a group's keys, at most LG_KEYS, in registers during a select);
//                            every CTA-wide step runs once for all G groups, so a sub-tile costs the barriers of one
//                            group. Keys are read from the staged arrays with coalesced loads; flags, votes and the
//                            per-member bandwidth sums follow, the sums gathered in shared memory over all tiles a CTA
//                            handles of one communicator and window (the grid is persistent).
//   k_reduce_large_deferred  the groups that are not complete and 32-bit clean (a missing member, a record in flight,
//                            invalid times, spreads beyond 32 bits): one CTA per listed group, 64-bit throughout, hang alerts.
#pragma once
#include "ccld_device.cuh"

namespace ccld {

// What k_large_stage leaves per group; every field is a maximum (minima are stored complemented), so zero is the
// neutral start. bits: 1 = some record disqualifies the group for the 32-bit path, 2 = the op set differs inside it.
struct LargeGroup { u64 kmax, n_kmin, ck; u32 n_emin, emax, xmax, bits; };
struct LargeLead { u64 brng; u32 bk, rounds, an, def, pad; };
// per-group values the flag pass reads back from shared memory
struct LargeScal { u64 ts, td; double bn, den; u32 emin, tmn, ms, md; u32 state, pad; };       // state: 1 group handled here, 2 analysed, 4 barrier

constexpr u32 LS_PITCH = LS_MEMBERS + 4;     // lanes (op counter 0..7, member 0..3) hit 32 distinct banks

__global__ void __launch_bounds__(LS_THREADS, 4) k_large_stage(const WinDesc* __restrict__ wd, const Tile* __restrict__ tiles, LargeGroup* __restrict__ grp, Registry R) {
  __shared__ u32 s_a[LARGE_SEQS * LS_PITCH], s_d[LARGE_SEQS * LS_PITCH];
  __shared__ LargeGroup s_part[LS_THREADS / 32][LARGE_SEQS];
  const Tile t = tiles[blockIdx.x];
  const WinDesc& D = wd[t.w];
  const u32 n = R.comm_n[t.c], m0 = blockIdx.y * LS_MEMBERS;
  if (m0 >= n) return;
  const RangeRow row = D.ranges[t.c];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const u32 j = lane & 7, pq = lane >> 3;                     // op counter of the tile, member of the quad
  const bool jvalid = j < t.count;
  const u32 so = t.seq_off + (jvalid ? j : 0u);
  const u32* __restrict__ perm = D.perm + row.slot0;
  const i64* __restrict__ c_te = D.t_enter; const i64* __restrict__ c_tx = D.t_exit;
  const u64* __restrict__ c_by = D.bytes; const u8* __restrict__ c_op = D.op;
  const u32* __restrict__ c_sc = D.send_chg; const u32* __restrict__ c_rc = D.recv_chg;
  // the group's first member gives the time base and the op set
  u32 bits = 0;
  i64 te0 = 0; u64 by0 = 0; u32 op0 = 0;
  {
    const u32 i0 = jvalid ? __ldg(perm + so) : NONE;
    if (i0 != NONE) { te0 = c_te[i0]; by0 = c_by[i0]; op0 = c_op[i0]; } else bits = 1;
  }
  const u64 base = (u64)te0 - 0x80000000ull;
  u32 emin = 0xFFFFFFFFu, emax = 0, xmax = 0; u64 kmax = 0, kmin = U64_MAX_, ck = 0;
  constexpr u32 PER_WARP = LS_MEMBERS / (LS_THREADS / 32);    // 64 members per warp, four at a time
  for (u32 it = 0; it < PER_WARP / 4; it += 4) {
    u32 idx[4]; i64 x[4], y[4]; u64 by[4]; u32 op[4], ch[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) { const u32 p = m0 + wid * PER_WARP + (it + q) * 4 + pq; idx[q] = (jvalid && p < n) ? __ldg(perm + (u64)p * row.n_seq + so) : NONE; }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 ix = idx[q] == NONE ? 0u : idx[q];
      x[q] = c_te[ix]; y[q] = c_tx[ix]; by[q] = c_by[ix]; op[q] = c_op[ix]; ch[q] = 0;
      if (c_sc != nullptr) { const u32 sc = c_sc[ix], rc = c_rc[ix]; ch[q] = sc > rc ? sc : rc; }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 pm = wid * PER_WARP + (it + q) * 4 + pq, p = m0 + pm;
      u32 a_lo = 0, d = 0;
      if (p < n) {
        if (idx[q] == NONE) { if (jvalid) bits |= 1; }
        else {
          const u64 ra = (u64)x[q] - base, rb = (u64)y[q] - base;
          a_lo = (u32)ra; const u32 b_lo = (u32)rb; d = b_lo - a_lo;
          if (((ra | rb) >> 32) != 0 || (x[q] | y[q]) < 0 || b_lo < a_lo) bits |= 1;     // beyond 32 bits, negative or in flight, exit before enter
          if (op[q] != op0 || by[q] != by0) bits |= 2;
          emin = min(emin, a_lo); emax = max(emax, a_lo); xmax = max(xmax, b_lo);
          const u64 k1 = ((u64)d << 32) | (u64)(NONE - p); kmax = k1 > kmax ? k1 : kmax;   // longest, then the lowest position
          const u64 k2 = ((u64)d << 32) | (u64)p; kmin = k2 < kmin ? k2 : kmin;            // shortest, then the lowest position
          const u64 k3 = ((u64)ch[q] << 32) | (u64)(NONE - p); ck = k3 > ck ? k3 : ck;     // most changes, then the lowest position
        }
      }
      s_a[j * LS_PITCH + pm] = a_lo; s_d[j * LS_PITCH + pm] = d;
    }
  }
  // the four members of a warp step meet by shuffles, the warps through shared memory; one thread per op counter merges
  // the CTA's part into the group's record
#pragma unroll
  for (int h = 8; h < 32; h <<= 1) {
    emin = min(emin, __shfl_xor_sync(0xFFFFFFFFu, emin, h)); emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, h));
    xmax = max(xmax, __shfl_xor_sync(0xFFFFFFFFu, xmax, h)); bits |= __shfl_xor_sync(0xFFFFFFFFu, bits, h);
    const u64 a = shfl_xor64(kmax, h); kmax = a > kmax ? a : kmax;
    const u64 b = shfl_xor64(kmin, h); kmin = b < kmin ? b : kmin;
    const u64 e = shfl_xor64(ck, h); ck = e > ck ? e : ck;
  }
  if (lane < LARGE_SEQS) { LargeGroup x; x.kmax = kmax; x.n_kmin = ~kmin; x.ck = ck; x.n_emin = ~emin; x.emax = emax; x.xmax = xmax; x.bits = bits; s_part[wid][lane] = x; }
  __syncthreads();
  if (threadIdx.x < t.count) {
    LargeGroup a = s_part[0][threadIdx.x];
    for (u32 w = 1; w < LS_THREADS / 32; ++w) {
      const LargeGroup x = s_part[w][threadIdx.x];
      a.kmax = x.kmax > a.kmax ? x.kmax : a.kmax; a.n_kmin = x.n_kmin > a.n_kmin ? x.n_kmin : a.n_kmin; a.ck = x.ck > a.ck ? x.ck : a.ck;
      a.n_emin = max(a.n_emin, x.n_emin); a.emax = max(a.emax, x.emax); a.xmax = max(a.xmax, x.xmax); a.bits |= x.bits;
    }
    LargeGroup* o = grp + (u64)blockIdx.x * LARGE_SEQS + threadIdx.x;
    atomicMax((ull*)&o->kmax, (ull)a.kmax); atomicMax((ull*)&o->n_kmin, (ull)a.n_kmin); atomicMax((ull*)&o->ck, (ull)a.ck);
    atomicMax(&o->n_emin, a.n_emin); atomicMax(&o->emax, a.emax); atomicMax(&o->xmax, a.xmax);
    if (a.bits) atomicOr(&o->bits, a.bits);
  }
  // keys leave group by group, members contiguous
  const u32 cnt = n - m0 < LS_MEMBERS ? n - m0 : (u32)LS_MEMBERS;
  for (u32 q = 0; q < t.count; ++q) {
    const u64 o = row.slot0 + (u64)(t.seq_off + q) * n + m0;
    for (u32 pm = threadIdx.x; pm < cnt; pm += LS_THREADS) { D.skey[o + pm] = s_a[q * LS_PITCH + pm]; D.dkey[o + pm] = s_d[q * LS_PITCH + pm]; }
  }
}

constexpr u32 LG_DIGIT = 8, LG_BINS = 1u << LG_DIGIT;      // radix digit of the selects; one histogram of LG_BINS bins per group

// The k-th smallest (0-based) of a group's keys, for every group of the sub-tile at once. A thread holds up to LG_KEYS keys
// of its own group g in registers (bit q of `have` says whether slot q holds one); `act` says whether the group takes
// part. Digits of LG_DIGIT bits, most significant first; the first digit starts at the highest bit of `bound`, the
// largest key of any group, so that it splits the keys as finely as 256 bins can, and a key that drops out of the
// running costs its thread next to nothing in the passes that follow. After a pass warp w scans and clears group w's
// histogram and names the digit that holds the k-th key. Histograms must be zero on entry and are zero again on return.
// All threads of the CTA call it.
__device__ __forceinline__ u32 large_select(const u32 (&v)[LG_KEYS], u32 have, bool act, u32 k, u32 bound, u32 G, u32 g,
                                            u32* __restrict__ s_hist, u32* __restrict__ s_pick, u32* __restrict__ s_krem) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x < G) s_krem[threadIdx.x] = k;
  u32* __restrict__ hist = s_hist + g * LG_BINS;
  u32 hi = 32 - (u32)__clz(bound | 1u);                      // bits still undecided: the result lies below 2^hi
  u32 prefix = 0;                                            // the decided bits, already in place
  u32 alive = act ? have : 0u;                               // my keys that still agree with the decided bits
  while (hi > 0) {
    const u32 sh = hi > LG_DIGIT ? hi - LG_DIGIT : 0u, w = hi - sh;       // this pass decides bits [sh, hi)
    const u32 dmask = (1u << w) - 1u;
    if (alive) {
#pragma unroll
      for (int q = 0; q < LG_KEYS; ++q) if ((alive >> q) & 1u) atomicAdd(&hist[(v[q] >> sh) & dmask], 1u);
    }
    __syncthreads();
    if (wid < G) {                                                               // warp w scans and clears group w's histogram
      u32 loc[8], sum = 0;
      const u32 kr = s_krem[wid];
#pragma unroll
      for (int q = 0; q < 8; ++q) { loc[q] = s_hist[wid * LG_BINS + lane * 8 + q]; sum += loc[q]; s_hist[wid * LG_BINS + lane * 8 + q] = 0; }
      u32 inc = sum;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) { const u32 o = __shfl_up_sync(0xFFFFFFFFu, inc, d); if (lane >= (u32)d) inc += o; }
      const u32 ex = inc - sum;
      if (kr >= ex && kr < inc) {
        u32 cum = ex;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (kr >= cum && kr < cum + loc[q]) { s_pick[wid] = lane * 8 + q; s_krem[wid] = kr - cum; }
          cum += loc[q];
        }
      }
    }
    __syncthreads();
    const u32 pick = s_pick[g];
    prefix |= pick << sh;
    if (alive) {                                             // few keys survive the first pass: most threads are done here
      u32 keep = 0;
#pragma unroll
      for (int q = 0; q < LG_KEYS; ++q) keep |= (((v[q] >> sh) & dmask) == pick ? 1u : 0u) << q;
      alive &= keep;
    }
    hi = sh;
  }
  return prefix;
}

// dynamic shared memory of k_reduce_large: per-member bandwidth sums of the largest communicator
inline size_t large_smem(u32 max_n) { return (size_t)8 * large_npad(max_n); }

__global__ void __launch_bounds__(LG_THREADS, 2) k_reduce_large(const WinDesc* __restrict__ wd, const Tile* __restrict__ tiles, u32 n_tiles,
                                                                 const LargeGroup* __restrict__ grp, TileSum* __restrict__ sums,
                                                                 Registry R, Params P, DeferList DL) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* s_bw = (double*)smem_raw;
  __shared__ u32 s_hist[LARGE_SEQS * LG_BINS];
  __shared__ LargeScal s_sc[LARGE_SEQS];
  __shared__ LargeLead s_lead[LARGE_SEQS];
  __shared__ u32 s_cnt[SC_COUNT];
  __shared__ u32 s_bound[2][LARGE_SEQS];
  __shared__ u32 s_pick[LARGE_SEQS], s_krem[LARGE_SEQS];
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u32 cur_w = NONE, cur_c = NONE, cur_rounds = 0;            // whose bandwidth sums shared memory holds
  const u32* cur_mem = nullptr; u32 cur_n = 0;
  for (u32 i = threadIdx.x; i < LARGE_SEQS * LG_BINS; i += LG_THREADS) s_hist[i] = 0;
  for (u32 ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
    const Tile t = tiles[ti];
    const WinDesc& D = wd[t.w];
    const u32 c = t.c, n = R.comm_n[c];
    const RangeRow row = D.ranges[c];
    const u32* __restrict__ mem = R.members + R.comm_moff[c];
    const u32 G = large_g(n), lgG = 31 - __clz(G);
    const u32 g = wid & (G - 1), pl = (wid >> lgG) * 32 + lane, MP = (LG_WARPS >> lgG) * 32;      // a warp works on one group, lanes on consecutive members
    const bool lead = pl == 0;
    const u64 G_all = D.n_groups;

    __syncthreads();                                          // the previous tile is done with shared memory
    if (t.w != cur_w || c != cur_c) {
      // another communicator or window: the sums shared memory holds go out
      if (cur_rounds) for (u32 p = threadIdx.x; p < cur_n; p += LG_THREADS) { atomicAdd(&R.bw_sum[cur_mem[p]], s_bw[p]); atomicAdd(&R.bw_cnt[cur_mem[p]], cur_rounds); }
      __syncthreads();
      cur_w = t.w; cur_c = c; cur_rounds = 0; cur_mem = mem; cur_n = n;
      for (u32 p = threadIdx.x; p < n; p += LG_THREADS) s_bw[p] = 0.0;
    }
    if (threadIdx.x < SC_COUNT) s_cnt[threadIdx.x] = 0;
    if (threadIdx.x < LARGE_SEQS) { LargeLead z = {0, NONE, 0, 0, 0, 0}; s_lead[threadIdx.x] = z; }
    u32 have = 0;
#pragma unroll
    for (int q = 0; q < LG_KEYS; ++q) have |= (pl + (u32)q * MP < n ? 1u : 0u) << q;

    for (u32 j0 = 0; j0 < t.count; j0 += G) {
      const bool gvalid = j0 + g < t.count;
      const u32 so = t.seq_off + j0 + (gvalid ? g : 0u);      // op-counter offset of my group inside the range
      const u64 slot = row.slot0 + (u64)so * n;               // first slot of my group (keys and flags, group-major)
      __syncthreads();                                        // the previous sub-tile's shared-memory values are no longer read
      // ---- what the staging pass left for the group; op and size of its first member ----
      const LargeGroup x = grp[(u64)ti * LARGE_SEQS + j0 + (gvalid ? g : 0u)];
      const u32 emin = ~x.n_emin, tmx = (u32)(x.kmax >> 32), tmn = (u32)(~x.n_kmin >> 32);
      u64 by0 = 0; u32 op0 = 0; i64 te0 = 0;
      const bool gok = gvalid && !(x.bits & 1);
      if (gok) { const u32 i0 = __ldg(D.perm + row.slot0 + so); by0 = D.bytes[i0]; op0 = D.op[i0]; te0 = D.t_enter[i0]; }
      const bool barrier = op0 == CCLD_OP_ALLREDUCE && by0 < P.barrier_bytes;
      const bool analysed = gok && !barrier && n >= P.min_group;
      double num, den; bus_factor(op0, n, &num, &den);
      const double bn = (double)by0 * num;
      if (lead) {
        s_bound[0][g] = analysed ? x.emax - emin : 0u; s_bound[1][g] = analysed ? tmx - tmn : 0u;
        if (gvalid && !gok) {                                 // set aside for the 64-bit kernel
          const u32 e = atomicAdd(DL.count, 1u);
          DL.entries[e] = ((u64)t.w << 32) | (u64)(row.group0 + so);
          s_lead[g].def += 1;
        }
        if (gok) {
          // everything of the per-op row that needs no order statistic
          const u64 kmin = ~x.n_kmin;
          const u64 gi_ = row.group0 + so;
          i64* __restrict__ gi = D.gi64 + gi_; u32* __restrict__ gu = D.gu32 + gi_;
          const u32 span = x.xmax - emin;
          gi[(u64)GI_E_MIN * G_all] = (i64)((u64)te0 - 0x80000000ull + emin); gi[(u64)GI_ARRIVAL_SKEW * G_all] = (i64)(u64)(x.emax - emin);
          gi[(u64)GI_T_MAX * G_all] = (i64)(u64)tmx; gi[(u64)GI_T_MIN * G_all] = (i64)(u64)tmn; gi[(u64)GI_SPAN * G_all] = (i64)(u64)span;
          gu[(u64)GU_RANK_TMIN * G_all] = mem[(u32)kmin]; gu[(u64)GU_RANK_TMAX * G_all] = mem[NONE - (u32)x.kmax];
          gu[(u64)GU_MAX_CHG * G_all] = (u32)(x.ck >> 32); gu[(u64)GU_RANK_MAX_CHG * G_all] = mem[NONE - (u32)x.ck];
          gu[(u64)GU_N_PRESENT * G_all] = n;
          const bool mismatch = (x.bits & 2) != 0;
          gu[(u64)GU_GFLAGS * G_all] = CCLD_G_COMPLETE | (barrier ? CCLD_G_BARRIER : 0) | (mismatch ? CCLD_G_OPSET_MISMATCH : 0) | (analysed ? CCLD_G_ANALYSED : 0);
          D.gbw[gi_] = span ? bn * rcp_newton((double)span * den) : 0.0;
          atomicAdd(&s_cnt[SC_COMP], 1u); atomicAdd(&s_cnt[SC_PRES], n);
          if (barrier) atomicAdd(&s_cnt[SC_BAR], 1u);
          if (analysed) { atomicAdd(&s_cnt[SC_AN], 1u); s_lead[g].an += 1; }
          if (mismatch) atomicAdd(&s_cnt[SC_MIS], 1u);
          if (!barrier) { LargeLead m = s_lead[g]; m.rounds += 1; best_merge(m.brng, m.bk, (u64)(tmx - tmn), so); s_lead[g] = m; }
        }
      }
      __syncthreads();
      u32 bs = 0, bd = 0;
      for (u32 q = 0; q < G; ++q) { bs = max(bs, s_bound[0][q]); bd = max(bd, s_bound[1][q]); }

      // ---- order statistics, all groups of the sub-tile side by side; a thread's keys sit in registers during a select ----
      u32 ms = 0, ds = 0, md = 0, dm = 0;
      if (__syncthreads_or(analysed)) {
        const u32 k = (n - 1) >> 1;
        u32 v[LG_KEYS];
        const u32* __restrict__ sk = D.skey + slot + pl; const u32* __restrict__ du = D.dkey + slot + pl;
#pragma unroll
        for (int q = 0; q < LG_KEYS; ++q) v[q] = (analysed && ((have >> q) & 1u)) ? sk[(u32)q * MP] - emin : 0u;
        ms = large_select(v, have, analysed, k, bs, G, g, s_hist, s_pick, s_krem);
#pragma unroll
        for (int q = 0; q < LG_KEYS; ++q) v[q] = __usad(v[q], ms, 0u);
        ds = large_select(v, have, analysed, k, bs, G, g, s_hist, s_pick, s_krem);
#pragma unroll
        for (int q = 0; q < LG_KEYS; ++q) v[q] = (analysed && ((have >> q) & 1u)) ? du[(u32)q * MP] - tmn : 0u;
        md = large_select(v, have, analysed, k, bd, G, g, s_hist, s_pick, s_krem);
#pragma unroll
        for (int q = 0; q < LG_KEYS; ++q) v[q] = __usad(v[q], md, 0u);
        dm = large_select(v, have, analysed, k, bd, G, g, s_hist, s_pick, s_krem);
        if (!analysed) { ms = ds = md = dm = 0; }
      }
      if (lead) {
        LargeScal z; z.ts = (u64)ds * P.k_milli; z.td = (u64)dm * P.k_milli; z.bn = bn; z.den = den;   // |x - med| * 1000 > k * MAD: both sides below 2^64
        z.emin = emin; z.tmn = tmn; z.ms = ms; z.md = md; z.state = (gok ? 1u : 0u) | (analysed ? 2u : 0u) | (barrier ? 4u : 0u); z.pad = 0;
        s_sc[g] = z;
        if (gok) {
          i64* __restrict__ gi = D.gi64 + row.group0 + so;
          gi[(u64)GI_MED_SKEW * G_all] = (i64)(u64)ms; gi[(u64)GI_MAD_SKEW * G_all] = (i64)(u64)ds;
          gi[(u64)GI_MED_DUR * G_all] = analysed ? (i64)((u64)tmn + md) : 0; gi[(u64)GI_MAD_DUR * G_all] = (i64)(u64)dm;
        }
      }
      __syncthreads();

      // ---- flags, votes, per-member bandwidth: a thread takes a member through the G groups ----
      u32 n_fs = 0, n_fd = 0;
      const u32 gcnt = t.count - j0 < G ? t.count - j0 : G;
      const u64 slot0 = row.slot0 + (u64)(t.seq_off + j0) * n;
      for (u32 q = 0; q < gcnt; ++q) {
        const LargeScal z = s_sc[q];                                           // the group's values stay in registers over my members
        if (!(z.state & 1)) continue;
        const u64 o0 = slot0 + (u64)q * n;
        for (u32 p = threadIdx.x; p < n; p += LG_THREADS) {                  // a member belongs to one thread: no two threads touch s_bw[p]
          const u32 d = D.dkey[o0 + p];
          u32 f = CCLD_F_NOT_ANALYSED;
          if (z.state & 2) {
            const u32 skw = D.skey[o0 + p] - z.emin, dd = d - z.tmn;
            const bool so_ = (u64)__usad(skw, z.ms, 0u) * 1000u > z.ts, shi = skw > z.ms;
            const bool dq = (u64)__usad(dd, z.md, 0u) * 1000u > z.td, dhi = dd > z.md;
            f = (so_ ? CCLD_F_SKEW_OUT : 0) | (dq ? CCLD_F_DUR_OUT : 0) | (shi ? CCLD_F_SKEW_HI : 0) | (dhi ? CCLD_F_DUR_HI : 0);
            if (so_) { ++n_fs; atomicAdd(&R.votes[(u64)mem[p] * 4 + (shi ? 0 : 1)], 1u); }
            if (dq) { ++n_fd; atomicAdd(&R.votes[(u64)mem[p] * 4 + (dhi ? 2 : 3)], 1u); }
          }
          D.flags[o0 + p] = (u8)f;
          if (!(z.state & 4) && d != 0) s_bw[p] += z.bn * rcp_newton1((double)d * z.den);
        }
      }
      n_fs = __reduce_add_sync(0xFFFFFFFFu, n_fs); n_fd = __reduce_add_sync(0xFFFFFFFFu, n_fd);
      if (lane == 0) { if (n_fs) atomicAdd(&s_cnt[SC_FS], n_fs); if (n_fd) atomicAdd(&s_cnt[SC_FD], n_fd); }
    }  // sub-tiles
    __syncthreads();
    for (u32 q = 0; q < LARGE_SEQS; ++q) cur_rounds += s_lead[q].rounds;
    if (threadIdx.x == 0) {
      TileSum ts; ts.best_rng = 0; ts.best_k = NONE; ts.n_rounds = 0; ts.n_an = 0; ts.pad = 0;
      for (u32 q = 0; q < LARGE_SEQS; ++q) { best_merge(ts.best_rng, ts.best_k, s_lead[q].brng, s_lead[q].bk); ts.n_rounds += s_lead[q].rounds; ts.n_an += s_lead[q].an; ts.pad += s_lead[q].def; }
      sums[ti] = ts;
      count_add(D.counters, C_COMPLETE, s_cnt[SC_COMP]); count_add(D.counters, C_BARRIER, s_cnt[SC_BAR]); count_add(D.counters, C_ANALYSED, s_cnt[SC_AN]);
      count_add(D.counters, C_MISMATCH, s_cnt[SC_MIS]); count_add(D.counters, C_PRESENT, s_cnt[SC_PRES]);
      count_add(D.counters, C_FLAG_SKEW, s_cnt[SC_FS]); count_add(D.counters, C_FLAG_DUR, s_cnt[SC_FD]);
    }
  }  // tiles of this CTA
  __syncthreads();
  if (cur_rounds) for (u32 p = threadIdx.x; p < cur_n; p += LG_THREADS) { atomicAdd(&R.bw_sum[cur_mem[p]], s_bw[p]); atomicAdd(&R.bw_cnt[cur_mem[p]], cur_rounds); }
}

// ------------------------------------------------------------------------------------------------
// the groups k_reduce_large set aside: one CTA per listed group; enter times and durations live in
// shared memory as 64-bit values, order statistics by most-significant-byte-first radix select
// ------------------------------------------------------------------------------------------------
constexpr int LARGE_DEF_THREADS = 1024;
constexpr int LARGE_DEF_GRID = 148;         // grid-stride over the list: one CTA per SM of a B200

// Reduction over the CTA (all threads call; blockDim.x a multiple of 32): warps reduce by shuffles, the first warp
// reduces the warps' partial results the same way, everyone reads the result from s_red[0].
template <class T, class Op>
__device__ T block_reduce(T v, Op op, T* s_red /*[32]*/) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) { T o = __shfl_xor_sync(0xFFFFFFFFu, v, d); v = op(v, o); }
  __syncthreads();
  if (lane == 0) s_red[wid] = v;
  __syncthreads();
  if (wid == 0) {
    T x = lane < nw ? s_red[lane] : Op::identity();
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) { T o = __shfl_xor_sync(0xFFFFFFFFu, x, d); x = op(x, o); }
    if (lane == 0) s_red[0] = x;
  }
  __syncthreads();
  return s_red[0];
}
struct OpMinU64 { __device__ u64 operator()(u64 a, u64 b) const { return a < b ? a : b; } static __device__ u64 identity() { return U64_MAX_; } };
struct OpMaxU64 { __device__ u64 operator()(u64 a, u64 b) const { return a > b ? a : b; } static __device__ u64 identity() { return 0; } };
struct OpMaxI64 { __device__ i64 operator()(i64 a, i64 b) const { return a > b ? a : b; } static __device__ i64 identity() { return INT64_MIN; } };
struct OpAddU32 { __device__ u32 operator()(u32 a, u32 b) const { return a + b; } static __device__ u32 identity() { return 0; } };
struct OpOrU32 { __device__ u32 operator()(u32 a, u32 b) const { return a | b; } static __device__ u32 identity() { return 0; } };
struct OpMinU32 { __device__ u32 operator()(u32 a, u32 b) const { return a < b ? a : b; } static __device__ u32 identity() { return NONE; } };

// k-th smallest (0-based) of key(i), i < n; max_key bounds the keys. All threads of the CTA call it.
template <class F>
__device__ u64 radix_select(F key, u32 n, u32 k, u64 max_key, u32* hist /*[256]*/, u32* s_pick /*[2]*/) {
  int top = max_key == 0 ? 0 : (63 - __clzll((long long)max_key)) >> 3;
  u64 prefix = 0, mask = 0; u32 krem = k;
  for (int b = top; b >= 0; --b) {
    for (u32 i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (u32 i = threadIdx.x; i < n; i += blockDim.x) {
      const u64 v = key(i);
      if ((v & mask) == prefix) {
        const u32 bin = (u32)(v >> (8 * b)) & 255u;
        const u32 m = __match_any_sync(__activemask(), bin);       // one atomic per distinct bin in the warp
        if ((threadIdx.x & 31) == (u32)(__ffs(m) - 1)) atomicAdd(&hist[bin], (u32)__popc(m));
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      u32 loc[8], sum = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) { loc[q] = hist[threadIdx.x * 8 + q]; sum += loc[q]; }
      u32 inc = sum;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) { u32 o = __shfl_up_sync(0xFFFFFFFFu, inc, d); if ((threadIdx.x & 31) >= (u32)d) inc += o; }
      u32 ex = inc - sum;
      if (krem >= ex && krem < inc) {
        u32 cum = ex;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (krem >= cum && krem < cum + loc[q]) { s_pick[0] = threadIdx.x * 8 + q; s_pick[1] = krem - cum; }
          cum += loc[q];
        }
      }
    }
    __syncthreads();
    prefix |= (u64)s_pick[0] << (8 * b); mask |= 0xFFull << (8 * b); krem = s_pick[1];
    __syncthreads();
  }
  return prefix;
}

__global__ void __launch_bounds__(LARGE_DEF_THREADS) k_reduce_large_deferred(const WinDesc* __restrict__ wd, DeferList DL, Registry R, Params P, i64 now) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ u64 s_red64[32];
  __shared__ u32 s_red32[32];
  __shared__ u32 s_hist[256];
  __shared__ u32 s_pick[2];
  const u32 total = *DL.count;
  for (u32 e = blockIdx.x; e < total; e += gridDim.x) {
    const u64 ent = DL.entries[e];
    const WinDesc& D = wd[(u32)(ent >> 32)];
    const u64 g = (u32)ent;
    u32 c;
    { // owner: the last communicator whose first group is <= g (communicators without groups share their successor's start)
      u32 lo = 0, hi = R.n_comms - 1;
      while (lo < hi) { const u32 mid = (lo + hi + 1) >> 1; if (D.ranges[mid].group0 <= g) lo = mid; else hi = mid - 1; }
      c = lo;
    }
    const RangeRow row = D.ranges[c];
    const u32 n = row.n, so = (u32)(g - row.group0);
    const u32* mem = R.members + R.comm_moff[c];
    u64* s_te = (u64*)smem_raw;
    u64* s_du = s_te + n;
    const u64 G = D.n_groups;
    __syncthreads();
    const u64 slot = row.slot0 + (u64)so * n;                      // flags, group-major
    const u32 seq = row.seq_lo + so;
    const u32* __restrict__ pm = D.perm + perm_at(row, so, 0);     // member p at pm[p * n_seq]
    const u64 pst = row.n_seq;
    // pass 1: gather, presence, first present member
    u32 npres = 0, first = NONE, stor = 0;
    for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) {
      const u32 idx = pm[p * pst];
      u64 te = 0, du = 0; u32 st = 0;
      if (idx != NONE) {
        const i64 x = D.t_enter[idx], y = D.t_exit[idx];
        st = 1 | (y == -1 ? 2 : ((x < 0 || y < x) ? 4 : 0));
        te = (u64)x; du = (u64)(y - x);
        ++npres; first = first == NONE ? p : first;
      }
      stor |= st; s_te[p] = te; s_du[p] = du;
    }
    npres = block_reduce(npres, OpAddU32(), s_red32);
    first = block_reduce(first, OpMinU32(), s_red32);
    stor = block_reduce(stor, OpOrU32(), s_red32);
    const bool have_first = first != NONE;
    u64 gbytes = 0; u32 gop = 0;
    if (have_first) { const u32 idx = pm[first * pst]; gbytes = D.bytes[idx]; gop = D.op[idx]; }
    const bool inflight = stor & 2, bad_time = stor & 4, complete = npres == n && !inflight && !bad_time;
    const bool barrier = have_first && gop == CCLD_OP_ALLREDUCE && gbytes < P.barrier_bytes;
    // pass 2: op-set check, rate column, in-flight age, extrema
    u32 mism = 0; i64 age = -1; u64 chk = 0;
    u64 e_min = U64_MAX_, tmax = 0, tmin = U64_MAX_; i64 x_max = INT64_MIN;
    for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) {
      const u32 idx = pm[p * pst];
      if (idx == NONE) continue;
      if (D.op[idx] != gop || D.bytes[idx] != gbytes) mism = 1;
      u32 ch = 0;
      if (D.send_chg != nullptr) { const u32 sc = D.send_chg[idx], rc = D.recv_chg[idx]; ch = sc > rc ? sc : rc; }
      const u64 ck = ((u64)ch << 32) | (u64)(NONE - p); chk = ck > chk ? ck : chk;
      const u64 te = s_te[p], du = s_du[p];
      if (D.t_exit[idx] == -1) { const i64 ag = now - (i64)te; age = ag > age ? ag : age; }
      e_min = te < e_min ? te : e_min; tmax = du > tmax ? du : tmax; tmin = du < tmin ? du : tmin;
      const i64 tx = (i64)(te + du); x_max = tx > x_max ? tx : x_max;
    }
    mism = block_reduce(mism, OpOrU32(), s_red32);
    age = block_reduce(age, OpMaxI64(), (i64*)s_red64);
    chk = block_reduce(chk, OpMaxU64(), s_red64);
    e_min = block_reduce(e_min, OpMinU64(), s_red64);
    tmax = block_reduce(tmax, OpMaxU64(), s_red64);
    tmin = block_reduce(tmin, OpMinU64(), s_red64);
    x_max = block_reduce(x_max, OpMaxI64(), (i64*)s_red64);
    u32 gfl = (mism ? CCLD_G_OPSET_MISMATCH : 0) | (barrier ? CCLD_G_BARRIER : 0) | (inflight ? CCLD_G_INFLIGHT : 0) |
              (bad_time ? CCLD_G_BAD_TIME : 0) | (complete ? CCLD_G_COMPLETE : CCLD_G_INCOMPLETE);
    const bool analysed = complete && !barrier && n >= P.min_group;
    const bool hang = !complete && inflight && age > P.hang_ns && !barrier;
    if (analysed) gfl |= CCLD_G_ANALYSED;
    if (hang) gfl |= CCLD_G_HANG_ALERT;

    if (!complete) {
      for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS)
        D.flags[slot + p] = pm[p * pst] == NONE ? (CCLD_F_NOT_ANALYSED | CCLD_F_MISSING) : CCLD_F_NOT_ANALYSED;
      if (threadIdx.x == 0) {
        if (hang) raise_alert(D, R.comm_id[c], seq, age);
        for (int q = 0; q < GI_COUNT; ++q) D.gi64[(u64)q * G + g] = 0;
        for (int q = 0; q < GU_COUNT; ++q) D.gu32[(u64)q * G + g] = 0;
        D.gu32[(u64)GU_N_PRESENT * G + g] = npres; D.gu32[(u64)GU_GFLAGS * G + g] = gfl; D.gbw[g] = 0.0;
        count_add(D.counters, C_INCOMPLETE, 1); count_add(D.counters, C_BARRIER, barrier); count_add(D.counters, C_MISMATCH, mism);
        count_add(D.counters, C_PRESENT, npres);
      }
      continue;
    }
    // positions of the extrema: lowest ring position among equals
    u32 pmax = NONE, pmin = NONE; u64 askew = 0;
    for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) {
      if (s_du[p] == tmax && p < pmax) pmax = p;
      if (s_du[p] == tmin && p < pmin) pmin = p;
      const u64 sk = s_te[p] - e_min; askew = sk > askew ? sk : askew;
    }
    pmax = block_reduce(pmax, OpMinU32(), s_red32);
    pmin = block_reduce(pmin, OpMinU32(), s_red32);
    askew = block_reduce(askew, OpMaxU64(), s_red64);
    const i64 span = x_max - (i64)e_min;
    double num, den; bus_factor(gop, n, &num, &den);
    const double bn = (double)gbytes * num;
    if (!barrier) {
      for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) { atomicAdd(&R.bw_sum[mem[p]], busbw(bn, den, (i64)s_du[p])); atomicAdd(&R.bw_cnt[mem[p]], 1u); }
    }
    u64 med_s = 0, mad_s = 0, med_d = 0, mad_d = 0; u32 n_fs = 0, n_fd = 0;
    if (analysed) {
      const u32 k = (n - 1) >> 1;
      med_s = radix_select([&](u32 i) { return s_te[i] - e_min; }, n, k, askew, s_hist, s_pick);
      { const u64 m = med_s, dmax = m > askew - m ? m : askew - m;
        mad_s = radix_select([&](u32 i) { return absdiff(s_te[i] - e_min, m); }, n, k, dmax, s_hist, s_pick); }
      med_d = tmin + radix_select([&](u32 i) { return s_du[i] - tmin; }, n, k, tmax - tmin, s_hist, s_pick);
      { const u64 m = med_d, dmax = (m - tmin) > (tmax - m) ? (m - tmin) : (tmax - m);
        mad_d = radix_select([&](u32 i) { return absdiff(s_du[i], m); }, n, k, dmax, s_hist, s_pick); }
      for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) {
        const u64 sk = s_te[p] - e_min, du = s_du[p];
        const bool so_ = mul_gt(absdiff(sk, med_s), 1000u, mad_s, P.k_milli), sh = sk > med_s;
        const bool dq = mul_gt(absdiff(du, med_d), 1000u, mad_d, P.k_milli), dh = du > med_d;
        D.flags[slot + p] = (so_ ? CCLD_F_SKEW_OUT : 0) | (dq ? CCLD_F_DUR_OUT : 0) | (sh ? CCLD_F_SKEW_HI : 0) | (dh ? CCLD_F_DUR_HI : 0);
        if (so_) { ++n_fs; atomicAdd(&R.votes[(u64)mem[p] * 4 + (sh ? 0 : 1)], 1u); }
        if (dq) { ++n_fd; atomicAdd(&R.votes[(u64)mem[p] * 4 + (dh ? 2 : 3)], 1u); }
      }
      n_fs = block_reduce(n_fs, OpAddU32(), s_red32);
      n_fd = block_reduce(n_fd, OpAddU32(), s_red32);
    } else {
      for (u32 p = threadIdx.x; p < n; p += LARGE_DEF_THREADS) D.flags[slot + p] = CCLD_F_NOT_ANALYSED;
    }
    if (threadIdx.x == 0) {
      D.gi64[(u64)GI_E_MIN * G + g] = (i64)e_min; D.gi64[(u64)GI_ARRIVAL_SKEW * G + g] = (i64)askew;
      D.gi64[(u64)GI_T_MAX * G + g] = (i64)tmax; D.gi64[(u64)GI_T_MIN * G + g] = (i64)tmin; D.gi64[(u64)GI_SPAN * G + g] = span;
      D.gi64[(u64)GI_MED_SKEW * G + g] = (i64)med_s; D.gi64[(u64)GI_MAD_SKEW * G + g] = (i64)mad_s;
      D.gi64[(u64)GI_MED_DUR * G + g] = (i64)med_d; D.gi64[(u64)GI_MAD_DUR * G + g] = (i64)mad_d;
      D.gu32[(u64)GU_RANK_TMIN * G + g] = mem[pmin]; D.gu32[(u64)GU_RANK_TMAX * G + g] = mem[pmax];
      D.gu32[(u64)GU_MAX_CHG * G + g] = (u32)(chk >> 32); D.gu32[(u64)GU_RANK_MAX_CHG * G + g] = mem[NONE - (u32)chk];
      D.gu32[(u64)GU_N_PRESENT * G + g] = npres; D.gu32[(u64)GU_GFLAGS * G + g] = gfl;
      D.gbw[g] = busbw(bn, den, span);
      count_add(D.counters, C_COMPLETE, 1); count_add(D.counters, C_BARRIER, barrier); count_add(D.counters, C_ANALYSED, analysed);
      count_add(D.counters, C_MISMATCH, mism); count_add(D.counters, C_PRESENT, npres);
      count_add(D.counters, C_FLAG_SKEW, n_fs); count_add(D.counters, C_FLAG_DUR, n_fd);
    }
  }
}

}  // namespace ccld
