// CCL-D decision-analyzer oracle: TEST INFRASTRUCTURE ONLY.
//
// A plain, sort-based C++17 statement of what the analyzer hot path computes,
// written from the paper's definitions (Sec. 4.1.2, Sec. 4.2.1 Eq. 1-3, Sec. 4.2.2 Eq. 4 and the
// hang decision tree of Fig. 6) and from the per-op statistics this repository adds to them
// (arrival skew, duration, bus bandwidth, lower-median / MAD outlier test, per-rank votes).
// One instance runs on one thread; independent instances (one per window) may run side by side on several host cores
// and their per-rank statistics add up (orc_add_rank_stats).
// It shares no code, header, table or helper with the CUDA library and must never be called by
// the product path: only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
//
// Nothing here is blocked, fused or reordered: every statistic is its textbook definition
// (std::sort, then index), every threshold test is an exact 128-bit integer comparison.
//
// Pins (tests/test_oracle_*.py): hand-built traces with known answers, the paper's limits of P
// (Sec. 4.2.2), the SendRate worked example (Sec. 4.1.2, Fig. 5), one trace per leaf of the hang
// decision tree, brute-force order statistics by counting, and invariants.
// orc_derive_rates (counter changes per op from raw probe samples) is pinned to the same worked example, to closed
// forms for a counter that advances every tick, to additivity over adjacent ops and to a numpy restatement.
// orc_opset_check (majority Operation Type Set of an op and the ranks that deviate) is pinned to hand cases and to a
// collections.Counter restatement.
// Tree communicators: the same-layer restriction is the paper's (Sec. 4.2.1); which member is named - the one lagging its
// layer's counters in a hang, the one changing more often than its layer in a slowdown - is this repository's rule
// ("parity unpinned"), pinned to hand cases.
// "Parity unpinned" against the paper: the bus-bandwidth factor and the median/MAD convention,
// because the paper defines neither (they are this repository's conventions, pinned only to
// closed forms and hand values).
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <map>
#include <string>
#include <unordered_map>
#include <vector>

typedef unsigned __int128 u128;
typedef int64_t i64;
typedef uint64_t u64;
typedef uint32_t u32;
typedef uint8_t u8;

namespace {

const u32 NONE = 0xFFFFFFFFu;

// op codes (the collectives the paper lists in Sec. 2.1, plus point-to-point and broadcast)
enum { OP_ALLREDUCE = 0, OP_ALLGATHER = 1, OP_REDUCESCATTER = 2, OP_ALLTOALL = 3, OP_SENDRECV = 4, OP_BROADCAST = 5 };

// per-slot flag byte
enum { F_SKEW_OUT = 1, F_DUR_OUT = 2, F_SKEW_HI = 4, F_DUR_HI = 8, F_MISSING = 64, F_NOT_ANALYSED = 128 };
// per-group flag word
enum { G_COMPLETE = 1, G_INCOMPLETE = 2, G_BARRIER = 4, G_OPSET_MISMATCH = 8, G_ANALYSED = 16, G_HANG_ALERT = 32, G_INFLIGHT = 64, G_BAD_TIME = 128 };
// input error bits
enum { E_UNKNOWN_COMM = 1, E_NOT_MEMBER = 2, E_SEQ_RANGE = 4, E_DUPLICATE = 8 };

struct Params {
  i64 tbase_init_ns; i64 theta_slow_milli, alpha_milli, beta_milli, m_max_rounds, m_max_ns, hang_ns;
  i64 barrier_bytes, slow_rep_threshold, k_milli, min_group, vote_rep_milli;
};

struct Comm {
  u32 id; u32 seq0; std::vector<u32> ranks; std::unordered_map<u32, u32> pos;
  std::vector<u32> layer;   // tree communicators: layer id of each member (empty: ring)
  // Eq. 1 state, carried across windows
  u64 rounds = 0; i64 t_first = 0; i64 sum_m = 0; u64 m = 0; u64 slow_count = 0;
};

struct GroupRow {
  u32 comm_idx, seq; u64 slot0;
  i64 e_min = 0, arrival_skew = 0, t_max = 0, t_min = 0, span = 0, med_skew = 0, mad_skew = 0, med_dur = 0, mad_dur = 0;
  u32 rank_tmin = 0, rank_tmax = 0, max_chg = 0, rank_max_chg = 0, n_present = 0, gflags = 0;
  double busbw = 0.0;
};

struct CommRow {
  u32 comm, n_rounds, sel_seq, cls, slow_detected, located, baseline_static, rate_source, root_comp, root_comm;
  u64 slow_count, rounds_total, m;
  i64 t_max, t_min, t_base;
  double R, P;
};

struct Alert { u32 comm, seq; i64 age; };

struct RankStat { u32 v[4] = {0, 0, 0, 0}; u32 ops = 0, bw_cnt = 0; double bw_sum = 0.0; };

struct Window {
  u64 n = 0;
  std::vector<u32> rank, comm, seq, send_chg, recv_chg; std::vector<u8> op, algo, proto; std::vector<u64> bytes; std::vector<i64> t_enter, t_exit;
  u32 n_frames = 0, n_channels = 0; std::vector<u32> f_rank, f_comm, f_seq, progress;
  bool analysed = false;
  // results
  std::vector<GroupRow> groups; std::vector<u8> flags; std::vector<u32> perm;
  std::vector<CommRow> comm_rows; std::vector<Alert> alerts;
  std::map<u32, std::pair<u32, u32>> range;   // comm_idx -> (seqlo, seqhi)
  std::map<u32, u64> first_group;             // comm_idx -> index of its first group
  u64 n_rejected = 0, n_complete = 0, n_incomplete = 0, n_barrier = 0, n_analysed = 0, n_flag_skew = 0, n_flag_dur = 0, n_mismatch = 0;
  u32 err = 0;
};

struct Oracle {
  Params p; std::vector<Comm> comms; std::unordered_map<u32, u32> comm_idx;
  std::map<u32, Window> windows; std::map<u32, RankStat> stats;
};

// Bus-bandwidth factor num/den per op (this repository's convention; n = communicator size).
void bus_factor(u8 op, u32 n, u64* num, u64* den) {
  switch (op) {
    case OP_ALLREDUCE: *num = 2 * (u64)(n - 1); *den = n; break;
    case OP_ALLGATHER: case OP_REDUCESCATTER: case OP_ALLTOALL: *num = n - 1; *den = n; break;
    default: *num = 1; *den = 1; break;
  }
}

double busbw(u64 bytes, u8 op, u32 n, i64 t) {
  if (t <= 0) return 0.0;
  u64 num, den; bus_factor(op, n, &num, &den);
  return ((double)bytes * (double)num) / ((double)t * (double)den);
}

// Lower median and lower-median absolute deviation by full sorts; flags by the exact integer test
// |x - med| * 1000 > k_milli * MAD.
void median_mad(const std::vector<i64>& x, i64 k_milli, i64* med, i64* mad, std::vector<u8>* out, std::vector<u8>* hi) {
  size_t n = x.size();
  std::vector<i64> s(x); std::sort(s.begin(), s.end());
  *med = s[(n - 1) / 2];
  std::vector<u64> d(n);
  for (size_t i = 0; i < n; ++i) d[i] = x[i] >= *med ? (u64)x[i] - (u64)*med : (u64)*med - (u64)x[i];
  std::vector<u64> ds(d); std::sort(ds.begin(), ds.end());
  u64 m = ds[(n - 1) / 2];
  *mad = (i64)m;
  out->assign(n, 0); hi->assign(n, 0);
  for (size_t i = 0; i < n; ++i) {
    (*out)[i] = ((u128)d[i] * 1000u > (u128)(u64)k_milli * m) ? 1 : 0;
    (*hi)[i] = x[i] > *med ? 1 : 0;
  }
}

void analyze_one(Oracle& o, Window& w, i64 now) {
  const Params& p = o.p;
  // ---- grouping: sort accepted records by (communicator, seq, ring position) ----
  struct Key { u32 c, s, pos; u64 rec; };
  std::vector<Key> keys; keys.reserve(w.n);
  for (u64 i = 0; i < w.n; ++i) {
    auto ci = o.comm_idx.find(w.comm[i]);
    if (ci == o.comm_idx.end()) { w.err |= E_UNKNOWN_COMM; ++w.n_rejected; continue; }
    Comm& c = o.comms[ci->second];
    // the op counters a communicator covers in this window: every record that names it with a
    // counter at or above its first one, whether or not the reporting rank turns out to be a member
    if (w.seq[i] >= c.seq0) {
      auto it = w.range.find(ci->second);
      if (it == w.range.end()) w.range[ci->second] = {w.seq[i], w.seq[i]};
      else { it->second.first = std::min(it->second.first, w.seq[i]); it->second.second = std::max(it->second.second, w.seq[i]); }
    }
    auto pi = c.pos.find(w.rank[i]);
    if (pi == c.pos.end()) { w.err |= E_NOT_MEMBER; ++w.n_rejected; continue; }
    if (w.seq[i] < c.seq0) { w.err |= E_SEQ_RANGE; ++w.n_rejected; continue; }
    keys.push_back(Key{ci->second, w.seq[i], pi->second, i});
  }
  std::stable_sort(keys.begin(), keys.end(), [](const Key& a, const Key& b) {
    if (a.c != b.c) return a.c < b.c;
    if (a.s != b.s) return a.s < b.s;
    return a.pos < b.pos;
  });
  u64 n_slots = 0;
  for (auto& r : w.range) {
    u32 n = (u32)o.comms[r.first].ranks.size();
    w.first_group[r.first] = w.groups.size();
    for (u64 s = r.second.first; s <= r.second.second; ++s) {
      GroupRow g; g.comm_idx = r.first; g.seq = (u32)s; g.slot0 = n_slots; n_slots += n;
      w.groups.push_back(g);
    }
  }
  w.perm.assign(n_slots, NONE);
  w.flags.assign(n_slots, F_MISSING | F_NOT_ANALYSED);
  for (const Key& k : keys) {
    const auto& r = w.range[k.c];
    u64 gi = w.first_group[k.c] + (k.s - r.first);
    u64 slot = w.groups[gi].slot0 + k.pos;
    if (w.perm[slot] != NONE) { w.err |= E_DUPLICATE; ++w.n_rejected; continue; }
    w.perm[slot] = (u32)k.rec;
  }

  // ---- per group ----
  for (GroupRow& g : w.groups) {
    Comm& c = o.comms[g.comm_idx];
    u32 n = (u32)c.ranks.size();
    const u32* rec = &w.perm[g.slot0];
    bool complete = true, inflight = false, bad_time = false, mismatch = false;
    u32 first = NONE;
    for (u32 q = 0; q < n; ++q) {
      if (rec[q] == NONE) { complete = false; continue; }
      ++g.n_present;
      w.flags[g.slot0 + q] = F_NOT_ANALYSED;
      u32 r = rec[q];
      if (first == NONE) first = r;
      else if (w.op[r] != w.op[first] || w.bytes[r] != w.bytes[first]) mismatch = true;
      if (w.t_exit[r] == -1) { inflight = true; complete = false; }
      else if (w.t_enter[r] < 0 || w.t_exit[r] < w.t_enter[r]) { bad_time = true; complete = false; }
    }
    // op type and size of the group are those of its lowest-position present member
    u8 gop = first == NONE ? 0 : w.op[first]; u64 gbytes = first == NONE ? 0 : w.bytes[first];
    bool barrier = first != NONE && gop == OP_ALLREDUCE && gbytes < (u64)p.barrier_bytes;
    if (mismatch) { g.gflags |= G_OPSET_MISMATCH; ++w.n_mismatch; }
    if (barrier) { g.gflags |= G_BARRIER; ++w.n_barrier; }
    if (inflight) g.gflags |= G_INFLIGHT;
    if (bad_time) g.gflags |= G_BAD_TIME;
    if (!complete) {
      g.gflags |= G_INCOMPLETE; ++w.n_incomplete;
      // hang detection (Sec. 4.2.1): an in-flight member older than the threshold, barriers filtered
      i64 age = -1;
      for (u32 q = 0; q < n; ++q)
        if (rec[q] != NONE && w.t_exit[rec[q]] == -1) age = std::max(age, now - w.t_enter[rec[q]]);
      if (inflight && age > p.hang_ns && !barrier) { g.gflags |= G_HANG_ALERT; w.alerts.push_back(Alert{c.id, g.seq, age}); }
      continue;
    }
    g.gflags |= G_COMPLETE; ++w.n_complete;
    std::vector<i64> te(n), dur(n), skew(n);
    i64 x_max = INT64_MIN;
    g.e_min = INT64_MAX; g.t_max = INT64_MIN; g.t_min = INT64_MAX;
    for (u32 q = 0; q < n; ++q) { te[q] = w.t_enter[rec[q]]; dur[q] = w.t_exit[rec[q]] - te[q]; g.e_min = std::min(g.e_min, te[q]); x_max = std::max(x_max, w.t_exit[rec[q]]); }
    g.max_chg = 0; g.rank_max_chg = c.ranks[0];
    bool have_chg = false;
    for (u32 q = 0; q < n; ++q) {
      skew[q] = te[q] - g.e_min;
      g.arrival_skew = std::max(g.arrival_skew, skew[q]);
      if (dur[q] > g.t_max) { g.t_max = dur[q]; g.rank_tmax = c.ranks[q]; }   // ties: lowest position
      if (dur[q] < g.t_min) { g.t_min = dur[q]; g.rank_tmin = c.ranks[q]; }
      u32 ch = 0;
      if (!w.send_chg.empty()) ch = std::max(w.send_chg[rec[q]], w.recv_chg[rec[q]]);
      if (!have_chg || ch > g.max_chg) { g.max_chg = ch; g.rank_max_chg = c.ranks[q]; have_chg = true; }
    }
    g.span = x_max - g.e_min;
    g.busbw = busbw(gbytes, gop, n, g.span);
    if (!barrier)
      for (u32 q = 0; q < n; ++q) { RankStat& st = o.stats[c.ranks[q]]; st.bw_sum += busbw(gbytes, gop, n, dur[q]); ++st.bw_cnt; }
    if (barrier || n < (u32)p.min_group) continue;
    // ---- median / MAD outlier test, votes ----
    g.gflags |= G_ANALYSED; ++w.n_analysed;
    std::vector<u8> so, sh, d_o, dh;
    median_mad(skew, p.k_milli, &g.med_skew, &g.mad_skew, &so, &sh);
    median_mad(dur, p.k_milli, &g.med_dur, &g.mad_dur, &d_o, &dh);
    for (u32 q = 0; q < n; ++q) {
      u8 f = 0;
      RankStat& st = o.stats[c.ranks[q]];
      ++st.ops;
      if (so[q]) { f |= F_SKEW_OUT; ++w.n_flag_skew; ++st.v[sh[q] ? 0 : 1]; }
      if (d_o[q]) { f |= F_DUR_OUT; ++w.n_flag_dur; ++st.v[dh[q] ? 2 : 3]; }
      if (sh[q]) f |= F_SKEW_HI;
      if (dh[q]) f |= F_DUR_HI;
      w.flags[g.slot0 + q] = f;
    }
  }

  // ---- window decision per communicator: Eq. 1-4 and the slow location rule ----
  for (auto& r : w.range) {
    Comm& c = o.comms[r.first];
    u64 g0 = w.first_group[r.first];
    u64 ng = (u64)r.second.second - r.second.first + 1;
    CommRow cr; std::memset(&cr, 0, sizeof cr);
    cr.comm = c.id; cr.sel_seq = NONE; cr.root_comp = NONE; cr.root_comm = NONE;
    const GroupRow* sel = nullptr;
    for (u64 k = 0; k < ng; ++k) {
      const GroupRow& g = w.groups[g0 + k];
      if (!(g.gflags & G_COMPLETE) || (g.gflags & G_BARRIER)) continue;
      ++cr.n_rounds;
      // Eq. 1: the first m rounds (at most m_max_rounds, all within m_max_ns of the first) feed the baseline
      if (c.m == 0) {
        if (c.rounds == 0) c.t_first = g.e_min;
        if (c.rounds == (u64)p.m_max_rounds || (c.rounds > 0 && g.e_min - c.t_first >= p.m_max_ns)) c.m = c.rounds;
        else c.sum_m += g.t_max;
      }
      ++c.rounds;
      // Eq. 2: round with the largest intra-round range, ties to the smallest seq
      if (sel == nullptr || g.t_max - g.t_min > sel->t_max - sel->t_min) sel = &g;
    }
    cr.baseline_static = c.m == 0;
    cr.t_base = c.m > 0 ? c.sum_m / (i64)c.m : p.tbase_init_ns;
    cr.rounds_total = c.rounds; cr.m = c.m;
    if (sel != nullptr) {
      cr.sel_seq = sel->seq; cr.t_max = sel->t_max; cr.t_min = sel->t_min;
      cr.R = (double)(cr.t_max - cr.t_base) / (double)cr.t_base;                       // Eq. 3
      cr.slow_detected = cr.t_max > cr.t_base && (u128)(u64)(cr.t_max - cr.t_base) * 1000u > (u128)(u64)p.theta_slow_milli * (u64)cr.t_base;
      if (cr.slow_detected) {
        ++c.slow_count;
        cr.located = c.slow_count > (u64)p.slow_rep_threshold;
        u64 num = (u64)(cr.t_max - cr.t_min), den = (u64)(cr.t_max - cr.t_base);
        cr.P = (double)num / (double)den;                                              // Eq. 4
        if ((u128)num * 1000u > (u128)(u64)p.beta_milli * den) cr.cls = 1;             // computation-slow
        else if ((u128)num * 1000u < (u128)(u64)p.alpha_milli * den) cr.cls = 2;       // communication-slow
        else cr.cls = 3;                                                               // mixed
        cr.root_comp = sel->rank_tmin;                  // minimal communication time
        if (sel->max_chg > 0) { cr.root_comm = sel->rank_max_chg; cr.rate_source = 0; }  // minimal rate = most changes
        else { cr.root_comm = sel->rank_tmax; cr.rate_source = 1; }
        if (!c.layer.empty()) {
          // tree (Sec. 4.2.1): update frequencies are comparable inside a layer only. The member with the most changes
          // above its layer's fewest; ties: the lowest position; every layer uniform: the rates name nobody.
          const u32 n = (u32)c.ranks.size();
          const u32* rec = &w.perm[sel->slot0];
          std::vector<u32> ch(n, 0);
          if (!w.send_chg.empty()) for (u32 q = 0; q < n; ++q) ch[q] = std::max(w.send_chg[rec[q]], w.recv_chg[rec[q]]);
          u32 best = 0; long at = -1;
          for (u32 q = 0; q < n; ++q) {
            u32 lmn = ch[q];
            for (u32 x = 0; x < n; ++x) if (c.layer[x] == c.layer[q]) lmn = std::min(lmn, ch[x]);
            if (ch[q] - lmn > best) { best = ch[q] - lmn; at = q; }
          }
          if (at >= 0) { cr.root_comm = c.ranks[at]; cr.rate_source = 0; }
          else { cr.root_comm = sel->rank_tmax; cr.rate_source = 1; }
        }
      }
    }
    cr.slow_count = c.slow_count;
    w.comm_rows.push_back(cr);
  }
  w.analysed = true;
}

}  // namespace

extern "C" {

void* orc_create(const i64* pv, int n) {
  if (n != 12) return nullptr;
  Oracle* o = new Oracle();
  std::memcpy(&o->p, pv, sizeof(Params));
  return o;
}
void orc_destroy(void* h) { delete (Oracle*)h; }

int orc_comm_register(void* h, u32 comm, const u32* ranks, u32 n, u32 seq0) {
  Oracle* o = (Oracle*)h;
  if (n == 0 || o->comm_idx.count(comm)) return -1;
  Comm c; c.id = comm; c.seq0 = seq0; c.ranks.assign(ranks, ranks + n);
  for (u32 i = 0; i < n; ++i) { if (c.pos.count(ranks[i])) return -1; c.pos[ranks[i]] = i; }
  o->comm_idx[comm] = (u32)o->comms.size();
  o->comms.push_back(std::move(c));
  return 0;
}

// Tree communicators (Sec. 4.2.1: only ranks of the same tree layer show consistent SendCount / RecvCount, so
// diagnostics that compare them are restricted to same-layer ranks). layer[i] belongs to the i-th registered member.
int orc_comm_set_layers(void* h, u32 comm, const u32* layer) {
  Oracle* o = (Oracle*)h;
  auto ci = o->comm_idx.find(comm);
  if (ci == o->comm_idx.end()) return -1;
  Comm& c = o->comms[ci->second];
  c.layer.assign(layer, layer + c.ranks.size());
  return 0;
}

int orc_upload(void* h, u32 wid, u64 n, const u32* rank, const u32* comm, const u32* seq, const u8* op, const u64* bytes,
               const i64* t_enter, const i64* t_exit, const u32* send_chg, const u32* recv_chg,
               u32 n_frames, const u32* f_rank, const u32* f_comm, const u32* f_seq, u32 n_channels, const u32* progress) {
  Oracle* o = (Oracle*)h;
  if (o->windows.count(wid)) return -1;
  Window& w = o->windows[wid];
  w.n = n;
  w.rank.assign(rank, rank + n); w.comm.assign(comm, comm + n); w.seq.assign(seq, seq + n); w.op.assign(op, op + n);
  w.bytes.assign(bytes, bytes + n); w.t_enter.assign(t_enter, t_enter + n); w.t_exit.assign(t_exit, t_exit + n);
  if (send_chg && recv_chg) { w.send_chg.assign(send_chg, send_chg + n); w.recv_chg.assign(recv_chg, recv_chg + n); }
  w.n_frames = n_frames; w.n_channels = n_channels;
  if (n_frames) {
    w.f_rank.assign(f_rank, f_rank + n_frames); w.f_comm.assign(f_comm, f_comm + n_frames); w.f_seq.assign(f_seq, f_seq + n_frames);
    w.progress.assign(progress, progress + (u64)n_frames * n_channels * 2);
  }
  return 0;
}

int orc_release(void* h, u32 wid) { return ((Oracle*)h)->windows.erase(wid) ? 0 : -1; }

int orc_analyze(void* h, u32 first, u32 count, i64 now) {
  Oracle* o = (Oracle*)h;
  for (u32 k = 0; k < count; ++k) {
    auto it = o->windows.find(first + k);
    if (it == o->windows.end() || it->second.analysed) return -1;
    analyze_one(*o, it->second, now);
  }
  return 0;
}

// sizes[0..11]: n_records, n_groups, n_slots, n_comm_rows, n_alerts, n_rejected, n_complete, n_incomplete, n_barrier,
// n_analysed, n_flag_skew, n_flag_dur; sizes[12] = n_opset_mismatch; sizes[13] = error bits
int orc_window_sizes(void* h, u32 wid, u64* s) {
  Oracle* o = (Oracle*)h; auto it = o->windows.find(wid);
  if (it == o->windows.end() || !it->second.analysed) return -1;
  Window& w = it->second;
  u64 v[14] = {w.n, w.groups.size(), w.perm.size(), w.comm_rows.size(), w.alerts.size(), w.n_rejected, w.n_complete,
               w.n_incomplete, w.n_barrier, w.n_analysed, w.n_flag_skew, w.n_flag_dur, w.n_mismatch, w.err};
  std::memcpy(s, v, sizeof v);
  return 0;
}

// Group table columns, one call copies all of them (arrays of length n_groups).
int orc_copy_groups(void* h, u32 wid, u32* comm, u32* seq, u64* slot0, i64* i9 /*[9][G]*/, u32* u6 /*[6][G]*/, double* bw) {
  Oracle* o = (Oracle*)h; Window& w = o->windows.at(wid);
  u64 G = w.groups.size();
  for (u64 i = 0; i < G; ++i) {
    const GroupRow& g = w.groups[i];
    comm[i] = o->comms[g.comm_idx].id; seq[i] = g.seq; slot0[i] = g.slot0;
    const i64 a[9] = {g.e_min, g.arrival_skew, g.t_max, g.t_min, g.span, g.med_skew, g.mad_skew, g.med_dur, g.mad_dur};
    for (int k = 0; k < 9; ++k) i9[k * G + i] = a[k];
    const u32 b[6] = {g.rank_tmin, g.rank_tmax, g.max_chg, g.rank_max_chg, g.n_present, g.gflags};
    for (int k = 0; k < 6; ++k) u6[k * G + i] = b[k];
    bw[i] = g.busbw;
  }
  return 0;
}

int orc_copy_slots(void* h, u32 wid, u8* flags, u32* perm) {
  Window& w = ((Oracle*)h)->windows.at(wid);
  std::memcpy(flags, w.flags.data(), w.flags.size());
  std::memcpy(perm, w.perm.data(), w.perm.size() * 4);
  return 0;
}

// Per communicator row: u32 x10, u64 x3, i64 x3, f64 x2 in separate arrays of length n_comm_rows.
int orc_copy_comm_rows(void* h, u32 wid, u32* u10, u64* u3, i64* i3, double* f2) {
  Window& w = ((Oracle*)h)->windows.at(wid);
  u64 n = w.comm_rows.size();
  for (u64 i = 0; i < n; ++i) {
    const CommRow& c = w.comm_rows[i];
    const u32 a[10] = {c.comm, c.n_rounds, c.sel_seq, c.cls, c.slow_detected, c.located, c.baseline_static, c.rate_source, c.root_comp, c.root_comm};
    for (int k = 0; k < 10; ++k) u10[k * n + i] = a[k];
    u3[0 * n + i] = c.slow_count; u3[1 * n + i] = c.rounds_total; u3[2 * n + i] = c.m;
    i3[0 * n + i] = c.t_max; i3[1 * n + i] = c.t_min; i3[2 * n + i] = c.t_base;
    f2[0 * n + i] = c.R; f2[1 * n + i] = c.P;
  }
  return 0;
}

int orc_copy_alerts(void* h, u32 wid, u32* comm, u32* seq, i64* age) {
  Window& w = ((Oracle*)h)->windows.at(wid);
  for (size_t i = 0; i < w.alerts.size(); ++i) { comm[i] = w.alerts[i].comm; seq[i] = w.alerts[i].seq; age[i] = w.alerts[i].age; }
  return 0;
}

// Cumulative per-rank statistics for ranks [0, n_ranks).
int orc_copy_rank_stats(void* h, u32 n_ranks, u32* votes /*[n][4]*/, u32* ops, u32* bw_cnt, double* bw_sum) {
  Oracle* o = (Oracle*)h;
  for (u32 r = 0; r < n_ranks; ++r) {
    auto it = o->stats.find(r);
    RankStat s; if (it != o->stats.end()) s = it->second;
    for (int k = 0; k < 4; ++k) votes[r * 4 + k] = s.v[k];
    ops[r] = s.ops; bw_cnt[r] = s.bw_cnt; bw_sum[r] = s.bw_sum;
  }
  return 0;
}

// Adds per-rank statistics gathered elsewhere (another oracle instance that analysed other windows) to this one's:
// votes, analysed-op counts and bandwidth sums are plain sums over windows, so windows analysed independently - each by
// its own single-threaded instance, possibly at the same time on different host cores - combine by addition.
int orc_add_rank_stats(void* h, u32 n_ranks, const u32* votes /*[n][4]*/, const u32* ops, const u32* bw_cnt, const double* bw_sum) {
  Oracle* o = (Oracle*)h;
  for (u32 r = 0; r < n_ranks; ++r) {
    if (ops[r] == 0 && bw_cnt[r] == 0 && !(votes[r * 4] | votes[r * 4 + 1] | votes[r * 4 + 2] | votes[r * 4 + 3])) continue;
    RankStat& s = o->stats[r];
    for (int k = 0; k < 4; ++k) s.v[k] += votes[r * 4 + k];
    s.ops += ops[r]; s.bw_cnt += bw_cnt[r]; s.bw_sum += bw_sum[r];
  }
  return 0;
}

// Suspects: kind 1 = straggler (late-arrival votes), kind 2 = slow link (long-duration votes);
// ordered by kind, then votes descending, then rank ascending. Returns the total count.
int orc_suspects(void* h, u32 cap, u32* kind, u32* rank, u32* votes, u32* ops, double* mean_bw) {
  Oracle* o = (Oracle*)h;
  struct S { u32 kind, rank, votes, ops; double bw; };
  std::vector<S> v;
  for (auto& kv : o->stats) {
    const RankStat& s = kv.second;
    if (s.ops == 0) continue;
    double bw = s.bw_cnt ? s.bw_sum / (double)s.bw_cnt : 0.0;
    if ((u64)s.v[0] * 1000u >= (u64)o->p.vote_rep_milli * s.ops) v.push_back(S{1, kv.first, s.v[0], s.ops, bw});
    if ((u64)s.v[2] * 1000u >= (u64)o->p.vote_rep_milli * s.ops) v.push_back(S{2, kv.first, s.v[2], s.ops, bw});
  }
  std::sort(v.begin(), v.end(), [](const S& a, const S& b) {
    if (a.kind != b.kind) return a.kind < b.kind;
    if (a.votes != b.votes) return a.votes > b.votes;
    return a.rank < b.rank;
  });
  for (size_t i = 0; i < v.size() && i < cap; ++i) { kind[i] = v[i].kind; rank[i] = v[i].rank; votes[i] = v[i].votes; ops[i] = v[i].ops; mean_bw[i] = v[i].bw; }
  return (int)v.size();
}

// Hang location (Sec. 4.2.2, Fig. 6) inside window `wid` for op (comm, seq).
// out[0..7] = class (1 H1, 2 H2, 3 H3), n_roots, n_not_entered, n_hung, n_not_hung, n_missing_frames, stuck_step, n_members
// min_total = the smallest per-rank sum of SendCount+RecvCount over channels (H3 only).
int orc_locate_hang(void* h, u32 wid, u32 comm, u32 seq, u32* out, u64* min_total, u32 cap, u32* roots) {
  Oracle* o = (Oracle*)h;
  auto wi = o->windows.find(wid); auto ci = o->comm_idx.find(comm);
  if (wi == o->windows.end() || ci == o->comm_idx.end()) return -1;
  Window& w = wi->second; Comm& c = o->comms[ci->second];
  u32 n = (u32)c.ranks.size();
  std::vector<u8> entered(n, 0), done(n, 0);
  for (u64 i = 0; i < w.n; ++i) {
    if (w.comm[i] != comm) continue;
    auto pi = c.pos.find(w.rank[i]); if (pi == c.pos.end()) continue;
    if (w.seq[i] >= seq) entered[pi->second] = 1;                 // operation counter reached the op
    if (w.seq[i] == seq && w.t_exit[i] != -1) done[pi->second] = 1;
  }
  std::vector<u32> r;
  u32 n_ne = 0, n_hung = 0, n_ok = 0, n_missing = 0, stuck = 0, cls;
  *min_total = 0;
  for (u32 q = 0; q < n; ++q) { if (!entered[q]) ++n_ne; if (done[q]) ++n_ok; else ++n_hung; }
  if (n_ne > 0) {                       // H1: ranks whose operation counter did not advance
    cls = 1; for (u32 q = 0; q < n; ++q) if (!entered[q]) r.push_back(c.ranks[q]);
  } else if (n_ok > 0) {                // H2: some ranks are not hung; they are the root cause
    cls = 2; for (u32 q = 0; q < n; ++q) if (done[q]) r.push_back(c.ranks[q]);
  } else {                              // H3: all hung; fewest SendCount/RecvCount
    cls = 3;
    std::vector<u64> tot(n, 0); std::vector<long> frame(n, -1);
    for (u32 f = 0; f < w.n_frames; ++f) {
      if (w.f_comm[f] != comm || w.f_seq[f] != seq) continue;
      auto pi = c.pos.find(w.f_rank[f]); if (pi == c.pos.end() || frame[pi->second] >= 0) continue;
      frame[pi->second] = f;
      for (u32 ch = 0; ch < w.n_channels; ++ch) tot[pi->second] += (u64)w.progress[((u64)f * w.n_channels + ch) * 2] + w.progress[((u64)f * w.n_channels + ch) * 2 + 1];
    }
    for (u32 q = 0; q < n; ++q) if (frame[q] < 0) ++n_missing;
    u64 mn = *std::min_element(tot.begin(), tot.end());
    long root = -1, first_min = -1;
    if (c.layer.empty()) {
      for (u32 q = 0; q < n; ++q) {
        if (tot[q] != mn) continue;
        if (first_min < 0) first_min = q;
        if (root < 0 && tot[(q + n - 1) % n] > mn) root = q;      // most upstream rank of a run of minima
      }
      if (root < 0) root = first_min;
    } else {
      // tree: a member is compared with its own layer only. Among the members that hold their layer's minimum while
      // another member of the layer is ahead, the one furthest behind its layer's maximum; ties: the lowest position.
      u64 best_lag = 0;
      for (u32 q = 0; q < n; ++q) {
        u64 lmn = tot[q], lmx = tot[q];
        for (u32 x = 0; x < n; ++x) if (c.layer[x] == c.layer[q]) { lmn = std::min(lmn, tot[x]); lmx = std::max(lmx, tot[x]); }
        if (tot[q] == lmn && lmx - lmn > best_lag) { best_lag = lmx - lmn; root = q; }
      }
      mn = root >= 0 ? tot[root] : 0;
    }
    if (root >= 0) r.push_back(c.ranks[root]);
    *min_total = mn;
    if (root >= 0 && frame[root] >= 0) {
      stuck = 0xFFFFFFFFu;
      for (u32 ch = 0; ch < w.n_channels; ++ch) stuck = std::min(stuck, w.progress[((u64)frame[root] * w.n_channels + ch) * 2 + 1]);
      if (w.n_channels == 0) stuck = 0;
    }
  }
  out[0] = cls; out[1] = (u32)r.size(); out[2] = n_ne; out[3] = n_hung; out[4] = n_ok; out[5] = n_missing; out[6] = stuck; out[7] = n;
  for (size_t i = 0; i < r.size() && i < cap; ++i) roots[i] = r[i];
  return 0;
}

// Operation Type Set (Sec. 4.1.2: algorithm, protocol, data size and operation name, constant during a communication;
// Sec. 4.2.2: inconsistent operations are what the not-hung ranks of leaf H2 point at). The two extra columns are
// attached per record; without them algorithm and protocol count as 0.
int orc_attach_opset(void* h, u32 wid, const u8* algo, const u8* proto) {
  Oracle* o = (Oracle*)h;
  auto wi = o->windows.find(wid);
  if (wi == o->windows.end()) return -1;
  Window& w = wi->second;
  w.algo.assign(algo, algo + w.n); w.proto.assign(proto, proto + w.n);
  return 0;
}

// For op (comm, seq): the most frequent (op, bytes, algo, proto) among the members that reported it - ties go to the
// tuple whose first holder stands earliest in the ring - and the members that carry another tuple, in ring order.
// out = {n_members, n_present, n_deviating, majority_count, op, algo, proto}; the first record of a member counts.
int orc_opset_check(void* h, u32 wid, u32 comm, u32 seq, u32* out, u64* bytes_out, u32 cap, u32* ranks) {
  Oracle* o = (Oracle*)h;
  auto wi = o->windows.find(wid); auto ci = o->comm_idx.find(comm);
  if (wi == o->windows.end() || ci == o->comm_idx.end()) return -1;
  Window& w = wi->second; Comm& c = o->comms[ci->second];
  const u32 n = (u32)c.ranks.size();
  std::vector<long> rec(n, -1);
  for (u64 i = 0; i < w.n; ++i) {
    if (w.comm[i] != comm || w.seq[i] != seq) continue;
    auto pi = c.pos.find(w.rank[i]);
    if (pi != c.pos.end() && rec[pi->second] < 0) rec[pi->second] = (long)i;
  }
  auto same = [&](long a, long b) {
    return w.op[a] == w.op[b] && w.bytes[a] == w.bytes[b] && (w.algo.empty() || (w.algo[a] == w.algo[b] && w.proto[a] == w.proto[b]));
  };
  u32 n_present = 0, best_cnt = 0; long best = -1;
  for (u32 p = 0; p < n; ++p) {
    if (rec[p] < 0) continue;
    ++n_present;
    u32 cnt = 0;
    for (u32 q = 0; q < n; ++q) if (rec[q] >= 0 && same(rec[p], rec[q])) ++cnt;
    if (cnt > best_cnt) { best_cnt = cnt; best = rec[p]; }      // positions ascend: the earliest holder wins ties
  }
  std::vector<u32> dev;
  for (u32 p = 0; p < n; ++p) if (rec[p] >= 0 && !same(rec[p], best)) dev.push_back(c.ranks[p]);
  out[0] = n; out[1] = n_present; out[2] = (u32)dev.size(); out[3] = best_cnt;
  out[4] = best >= 0 ? w.op[best] : 0; out[5] = best >= 0 && !w.algo.empty() ? w.algo[best] : 0; out[6] = best >= 0 && !w.proto.empty() ? w.proto[best] : 0;
  *bytes_out = best >= 0 ? w.bytes[best] : 0;
  for (size_t i = 0; i < dev.size() && i < cap; ++i) ranks[i] = dev[i];
  return 0;
}

// SendRate / RecvRate inputs from raw probe samples (Sec. 4.1.2: the rate is the reciprocal of the number of changes
// of SendCount / RecvCount seen by a probe that samples at a fixed period; Sec. 5.2 step 2: the diagnostic thread
// derives it from the counters). Rank r's samples are ticks [tick_off[r], tick_off[r+1]) in time order. For every
// record, the number of that rank's ticks k (not the rank's first) with t_enter < t_k <= t_end whose counter differs
// from the previous tick's; t_end = t_exit, or unbounded while the op is in flight (t_exit = -1).
void orc_derive_rates(u64 n_rec, const u32* rank, const i64* t_enter, const i64* t_exit, u32 n_ranks, const u64* tick_off,
                      const i64* tick_ns, const u32* send_count, const u32* recv_count, u32* send_chg, u32* recv_chg) {
  for (u64 i = 0; i < n_rec; ++i) {
    u32 s = 0, r = 0;
    if (rank[i] < n_ranks) {
      for (u64 k = tick_off[rank[i]] + 1; k < tick_off[rank[i] + 1]; ++k) {
        if (tick_ns[k] <= t_enter[i]) continue;
        if (t_exit[i] != -1 && tick_ns[k] > t_exit[i]) continue;
        if (send_count[k] != send_count[k - 1]) ++s;
        if (recv_count[k] != recv_count[k - 1]) ++r;
      }
    }
    send_chg[i] = s; recv_chg[i] = r;
  }
}

}  // extern "C"
