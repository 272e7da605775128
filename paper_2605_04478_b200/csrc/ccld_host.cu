// Host side of libccld: context, communicator registry, window upload, launch sequencing and result
// read-back. No analysis arithmetic lives here; every step of the hot path is a kernel in
// ccld_kernels.cuh.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>
#include <memory>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "ccld_kernels.cuh"
#include "ccld_rates.cuh"
#include "ccld_opset.cuh"

using namespace ccld;

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

struct Block { void* p = nullptr; size_t bytes = 0; };

struct CommHost {
  u32 id, seq0; std::vector<u32> ranks;
  u8 algo = 0;                      // 0 ring, 1 tree
  std::vector<u32> head;            // tree: lowest position of a member's layer (empty until the layers are set)
  const u32* d_head = nullptr;      // device copy inside the registry block
};

// Device blocks are recycled through a free list so that steady-state analysis allocates nothing.
struct Pool {
  std::vector<Block> free_list;
  Block get(size_t bytes, cudaError_t* err) {
    bytes = align_up(std::max<size_t>(bytes, ALIGN));
    int best = -1;
    for (size_t i = 0; i < free_list.size(); ++i)
      if (free_list[i].bytes >= bytes && free_list[i].bytes <= 2 * bytes + (1u << 20) && (best < 0 || free_list[i].bytes < free_list[best].bytes)) best = (int)i;
    if (best >= 0) { Block b = free_list[best]; free_list.erase(free_list.begin() + best); *err = cudaSuccess; return b; }
    Block b; b.bytes = bytes;
    *err = cudaMalloc(&b.p, bytes);
    if (*err != cudaSuccess) {                 // give cached blocks back to the driver and retry once
      for (auto& f : free_list) cudaFree(f.p);
      free_list.clear();
      *err = cudaMalloc(&b.p, bytes);
      if (*err != cudaSuccess) { b.p = nullptr; b.bytes = 0; }
    }
    return b;
  }
  void put(Block b) { if (b.p) free_list.push_back(b); }
  void clear() { for (auto& f : free_list) cudaFree(f.p); free_list.clear(); }
};

struct Shared {                                 // a pooled block shared by the windows of one batch
  Pool* pool; Block b;
  Shared(Pool* p, Block blk) : pool(p), b(blk) {}
  ~Shared() { pool->put(b); }
};

struct WindowHost {
  u32 id = 0; u64 n_rec = 0; bool owns = false; Block own;
  WinDesc d;                                    // device pointers
  u32 n_frames = 0, n_channels = 0;
  const u32 *f_rank = nullptr, *f_comm = nullptr, *f_seq = nullptr, *progress = nullptr;
  const u8 *algo = nullptr, *proto = nullptr; bool owns_opset = false; Block opset_own;   // Operation Type Set columns
  bool analysed = false;
  std::shared_ptr<Shared> plan_blk, res_blk;
  WinDesc* d_desc = nullptr;                    // this window's descriptor on the device
  u64 totals[T_COUNT];
  WindowHost() { std::memset(&d, 0, sizeof d); std::memset(totals, 0, sizeof totals); }
};

// A batch that was enqueued on totals the host expected instead of waiting for the plan: its actual totals arrive in
// pinned memory behind the batch's kernels and are checked at the next call that synchronizes anyway.
struct PendingBatch { u32 first = 0, n = 0; i64 now = 0; u64* h_tot = nullptr; size_t h_bytes = 0; };
// Totals of the last batches that were planned with a wait, by shape (record count of every window).
struct ShapeEntry { std::vector<u64> n_rec; std::vector<u64> totals; };
constexpr size_t SHAPE_CACHE = 4;

constexpr u32 TIMER_RING = 32;
constexpr int TIMER_PAIRS = CCLD_K_KINDS + 1;          // the layout kernel runs twice per call
struct TimerSlot { cudaEvent_t a[TIMER_PAIRS], b[TIMER_PAIRS]; int kind[TIMER_PAIRS]; int n = 0; };

}  // namespace

struct ccld_ctx {
  ccld_params params; Params dp; int device = 0; cudaStream_t stream = nullptr;
  std::vector<CommHost> comms; std::unordered_map<u32, u32> comm_idx;
  bool finalized = false; u32 n_ranks = 0, max_n = 0, max_large_n = 0; u64 sum_n = 0; size_t large_smem = 0; u32 n_sms = 148;
  Block reg_blk, misc_blk; Registry reg; size_t stats_off = 0, stats_bytes = 0;
  const TreeRef* d_trees = nullptr; u32 n_trees = 0;     // tree communicators whose layers are known
  std::map<u32, WindowHost> windows;
  Pool pool; std::string err;
  u64* h_pinned = nullptr; size_t h_pinned_bytes = 0;
  std::vector<PendingBatch> pending; std::vector<std::pair<u64*, size_t>> pinned_free; std::vector<ShapeEntry> shapes;
  u32* d_poison = nullptr; int speculate = 1;
  // optional per-kernel timing: a ring of event pairs, harvested lazily
  bool timing = false; std::vector<TimerSlot> ring; u32 ring_next = 0;
  double t_ms[CCLD_K_KINDS]; u64 t_launches[CCLD_K_KINDS];
  ccld_ctx() { std::memset(&reg, 0, sizeof reg); std::memset(t_ms, 0, sizeof t_ms); std::memset(t_launches, 0, sizeof t_launches); }
};

namespace {

int fail(ccld_ctx* c, int code, const std::string& msg) { if (c) c->err = msg; return code; }

#define CK(call)                                                                                   \
  do { cudaError_t e_ = (call);                                                                    \
       if (e_ != cudaSuccess) return fail(ctx, e_ == cudaErrorMemoryAllocation ? CCLD_ERR_NOMEM : CCLD_ERR_CUDA, \
                                          std::string(#call) + ": " + cudaGetErrorString(e_)); } while (0)

int ensure_pinned(ccld_ctx* ctx, size_t bytes) {
  if (ctx->h_pinned_bytes >= bytes) return CCLD_OK;
  if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
  ctx->h_pinned = nullptr; ctx->h_pinned_bytes = 0;
  CK(cudaMallocHost((void**)&ctx->h_pinned, bytes));
  ctx->h_pinned_bytes = bytes;
  return CCLD_OK;
}

// Adds the elapsed times of a slot's finished event pairs to the sums (waits for the last one).
void timer_harvest(ccld_ctx* ctx, TimerSlot& s) {
  for (int i = 0; i < s.n; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(s.b[i]) == cudaSuccess && cudaEventElapsedTime(&ms, s.a[i], s.b[i]) == cudaSuccess) {
      ctx->t_ms[s.kind[i]] += ms; ctx->t_launches[s.kind[i]] += 1;
    }
  }
  s.n = 0;
}
TimerSlot* timer_begin(ccld_ctx* ctx) {
  if (!ctx->timing) return nullptr;
  TimerSlot& s = ctx->ring[ctx->ring_next++ % TIMER_RING];
  timer_harvest(ctx, s);
  return &s;
}
// A named range for timeline tools (a no-op unless one is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete; NvtxRange& operator=(const NvtxRange&) = delete;
};
const char* const STAGE_NAMES[CCLD_K_KINDS] = {"ccld: op-counter ranges", "ccld: layout", "ccld: slot scatter", "ccld: reduce (up to 128 ranks)",
                                               "ccld: reduce (129 to 1024 ranks)", "ccld: reduce (more than 1024 ranks)", "ccld: window decision"};

struct TimedLaunch {                                     // a named range and, when timing is on, an event pair around one launch
  NvtxRange r; TimerSlot* s; cudaStream_t st; int i;
  TimedLaunch(TimerSlot* slot, int kind, cudaStream_t stream) : r(STAGE_NAMES[kind]), s(slot), st(stream), i(-1) {
    if (s && s->n < TIMER_PAIRS) { i = s->n++; s->kind[i] = kind; cudaEventRecord(s->a[i], st); }
  }
  ~TimedLaunch() { if (i >= 0) cudaEventRecord(s->b[i], st); }
};

// Layout of the scratch block used by get_verdict and locate_hang.
struct MiscLayout { size_t sus_a, sus_b, alerts, count, entered, done, frame, roots, tot, hang_out, total; };
MiscLayout misc_layout(u32 n_ranks, u32 max_n) {
  MiscLayout L; size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up(off + std::max<size_t>(b, 1)); return o; };
  L.sus_a = take(2ull * n_ranks * sizeof(ccld_suspect)); L.sus_b = take(2ull * n_ranks * sizeof(ccld_suspect));
  L.alerts = take(CCLD_MAX_ALERTS_PER_WINDOW * sizeof(ccld_hang_alert)); L.count = take(16);
  L.entered = take(max_n); L.done = take(max_n); L.frame = take(max_n * 4ull); L.roots = take(max_n * 4ull);
  L.tot = take(max_n * 8ull); L.hang_out = take(sizeof(ccld_hang_verdict));
  L.total = off;
  return L;
}

// Builds the device tables of the communicator registry and the per-rank statistics.
int finalize_registry(ccld_ctx* ctx) {
  if (ctx->finalized) return CCLD_OK;
  const u32 nc = (u32)ctx->comms.size();
  if (nc == 0) return fail(ctx, CCLD_ERR_STATE, "no communicator registered");
  u32 max_rank = 0; u64 sum_n = 0; u32 max_n = 0, max_large = 0;
  for (auto& c : ctx->comms) {
    for (u32 r : c.ranks) max_rank = std::max(max_rank, r);
    sum_n += c.ranks.size(); max_n = std::max<u32>(max_n, (u32)c.ranks.size());
    if (c.ranks.size() > MID_N) max_large = std::max<u32>(max_large, (u32)c.ranks.size());
  }
  const u32 nr = max_rank + 1;
  u32 hsize = 16; while (hsize < 2 * nc) hsize <<= 1;
  if (nc >= (1u << (32 - RANK_TAB_POS_BITS))) return fail(ctx, CCLD_ERR_CAPACITY, "too many communicators");
  std::vector<uint4> hash(hsize, make_uint4(0, NONE, 0, 0));
  std::vector<u32> comm_id(nc), comm_n(nc), comm_seq0(nc), members; std::vector<u64> moff(nc);
  std::vector<u32> rank_ptr(nr + 1, 0);
  members.reserve(sum_n);
  for (u32 i = 0; i < nc; ++i) {
    const CommHost& c = ctx->comms[i];
    comm_id[i] = c.id; comm_n[i] = (u32)c.ranks.size(); comm_seq0[i] = c.seq0; moff[i] = members.size();
    members.insert(members.end(), c.ranks.begin(), c.ranks.end());
    u32 h = (c.id * 2654435761u) & (hsize - 1);
    while (hash[h].y != NONE) h = (h + 1) & (hsize - 1);
    hash[h] = make_uint4(c.id, i, c.seq0, (u32)c.ranks.size());
    for (u32 r : c.ranks) ++rank_ptr[r + 1];
  }
  for (u32 r = 0; r < nr; ++r) rank_ptr[r + 1] += rank_ptr[r];
  std::vector<u32> ent_comm(sum_n), ent_pos(sum_n), fill(rank_ptr.begin(), rank_ptr.end() - 1);
  for (u32 i = 0; i < nc; ++i)
    for (u32 p = 0; p < ctx->comms[i].ranks.size(); ++p) { u32 r = ctx->comms[i].ranks[p]; ent_comm[fill[r]] = i; ent_pos[fill[r]] = p; ++fill[r]; }
  // inline (communicator id, index << 13 | position) pairs per rank, RANK_TAB_K of them in two uint4
  std::vector<u32> rank_tab((size_t)nr * 2 * RANK_TAB_K, NONE);
  for (u32 r = 0; r < nr; ++r) {
    const u32 cnt = rank_ptr[r + 1] - rank_ptr[r];
    const u32 inl = cnt <= (u32)RANK_TAB_K ? cnt : (u32)RANK_TAB_K - 1;
    for (u32 k = 0; k < inl; ++k) {
      const u32 ci = ent_comm[rank_ptr[r] + k];
      rank_tab[((size_t)r * RANK_TAB_K + k) * 2] = ctx->comms[ci].id;
      rank_tab[((size_t)r * RANK_TAB_K + k) * 2 + 1] = (ci << RANK_TAB_POS_BITS) | ent_pos[rank_ptr[r] + k];
    }
    if (cnt > (u32)RANK_TAB_K) rank_tab[((size_t)r * RANK_TAB_K + RANK_TAB_K - 1) * 2 + 1] = RANK_TAB_OVERFLOW;
  }

  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  const size_t o_hash = take(hsize * sizeof(uint4)), o_rtab = take(rank_tab.size() * 4), o_id = take(nc * 4), o_n = take(nc * 4), o_s0 = take(nc * 4), o_moff = take(nc * 8),
               o_mem = take(sum_n * 4), o_ptr = take((nr + 1) * 4ull), o_ec = take(sum_n * 4), o_ep = take(sum_n * 4);
  std::vector<size_t> o_head(nc, 0);
  u32 n_trees = 0;
  for (u32 i = 0; i < nc; ++i) if (!ctx->comms[i].head.empty()) { o_head[i] = take(ctx->comms[i].head.size() * 4); ++n_trees; }
  const size_t o_trees = take(std::max<u32>(n_trees, 1) * sizeof(TreeRef));
  const size_t o_stats = off;
  const size_t o_state = take(nc * sizeof(CommState)), o_votes = take(nr * 16ull), o_ops = take(nr * 4ull), o_cnt = take(nr * 4ull), o_bw = take(nr * 8ull);
  const size_t stats_end = off, o_poison = take(256);
  cudaError_t e;
  ctx->reg_blk = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "registry allocation failed");
  char* base = (char*)ctx->reg_blk.p;
  cudaStream_t st = ctx->stream;
  CK(cudaMemcpyAsync(base + o_hash, hash.data(), hsize * sizeof(uint4), cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_rtab, rank_tab.data(), rank_tab.size() * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_id, comm_id.data(), nc * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_n, comm_n.data(), nc * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_s0, comm_seq0.data(), nc * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_moff, moff.data(), nc * 8, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_mem, members.data(), sum_n * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_ptr, rank_ptr.data(), (nr + 1) * 4ull, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_ec, ent_comm.data(), sum_n * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(base + o_ep, ent_pos.data(), sum_n * 4, cudaMemcpyHostToDevice, st));
  for (u32 i = 0; i < nc; ++i) {
    CommHost& c = ctx->comms[i];
    if (c.head.empty()) continue;
    CK(cudaMemcpyAsync(base + o_head[i], c.head.data(), c.head.size() * 4, cudaMemcpyHostToDevice, st));
    c.d_head = (const u32*)(base + o_head[i]);
  }
  std::vector<TreeRef> trees;
  for (u32 i = 0; i < nc; ++i) if (ctx->comms[i].d_head) { TreeRef t; t.c = i; t.pad = 0; t.head = ctx->comms[i].d_head; trees.push_back(t); }
  if (n_trees) CK(cudaMemcpyAsync(base + o_trees, trees.data(), n_trees * sizeof(TreeRef), cudaMemcpyHostToDevice, st));
  ctx->d_trees = (const TreeRef*)(base + o_trees); ctx->n_trees = n_trees;
  CK(cudaMemsetAsync(base + o_stats, 0, off - o_stats, st));
  CK(cudaStreamSynchronize(st));              // the host vectors above go out of scope
  Registry& R = ctx->reg;
  R.n_comms = nc; R.hash_mask = hsize - 1; R.n_ranks = nr; R.pad = 0;
  R.hash = (const uint4*)(base + o_hash); R.rank_tab = (const uint4*)(base + o_rtab); R.comm_id = (const u32*)(base + o_id); R.comm_n = (const u32*)(base + o_n);
  R.comm_seq0 = (const u32*)(base + o_s0); R.comm_moff = (const u64*)(base + o_moff); R.members = (const u32*)(base + o_mem);
  R.rank_ptr = (const u32*)(base + o_ptr); R.ent_comm = (const u32*)(base + o_ec); R.ent_pos = (const u32*)(base + o_ep);
  R.state = (CommState*)(base + o_state); R.votes = (u32*)(base + o_votes); R.ops = (u32*)(base + o_ops);
  R.bw_cnt = (u32*)(base + o_cnt); R.bw_sum = (double*)(base + o_bw);
  ctx->stats_off = o_stats; ctx->stats_bytes = stats_end - o_stats; ctx->d_poison = (u32*)(base + o_poison);
  ctx->n_ranks = nr; ctx->max_n = max_n; ctx->max_large_n = max_large; ctx->sum_n = sum_n;

  // scratch for suspects, alert ordering and hang location
  ctx->misc_blk = ctx->pool.get(misc_layout(nr, max_n).total, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "scratch allocation failed");

  CK(cudaFuncSetAttribute(k_reduce_mid, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mid_smem_bytes(2 * WARP_N)));
  CK(cudaFuncSetAttribute(k_seq_range, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)range_smem_bytes(RANGE_DIRECT)));
  if (max_large) {
    ctx->large_smem = large_smem(max_large);
    CK(cudaFuncSetAttribute(k_reduce_large, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->large_smem));
    CK(cudaFuncSetAttribute(k_reduce_large_deferred, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(16ull * max_large)));
  }
  ctx->finalized = true;
  return CCLD_OK;
}

void drop_results(WindowHost& w) {
  w.analysed = false; w.plan_blk.reset(); w.res_blk.reset(); w.d_desc = nullptr;
  std::memset(w.totals, 0, sizeof w.totals);
}

int analyze_batch(ccld_ctx* ctx, u32 first_window, u32 n_windows, i64 now_ns, bool may_speculate);

u64* pinned_get(ccld_ctx* ctx, size_t bytes, size_t* got) {
  for (size_t i = 0; i < ctx->pinned_free.size(); ++i)
    if (ctx->pinned_free[i].second >= bytes) { auto p = ctx->pinned_free[i]; ctx->pinned_free.erase(ctx->pinned_free.begin() + i); *got = p.second; return p.first; }
  u64* p = nullptr;
  if (cudaMallocHost((void**)&p, bytes) != cudaSuccess) return nullptr;
  *got = bytes;
  return p;
}

// Brings the batches that were enqueued on expected totals to a definite state: waits for the stream, reads the totals
// their plans really found, and analyses again - this time waiting for the plan - every batch from the first one whose
// expectation failed (that batch and all later ones gave up on the device without touching any state, so the order of
// the windows is kept). Every call that hands out results or changes state goes through here first.
int settle(ccld_ctx* ctx) {
  if (ctx->pending.empty()) return CCLD_OK;
  CK(cudaSetDevice(ctx->device));
  CK(cudaStreamSynchronize(ctx->stream));
  std::vector<PendingBatch> todo;
  todo.swap(ctx->pending);
  bool failed = false;
  int rc = CCLD_OK;
  for (PendingBatch& b : todo) {
    for (u32 k = 0; k < b.n && !failed; ++k) if (b.h_tot[(size_t)k * T_COUNT + T_FAILED] == FAILED_EXPECT) failed = true;
    ctx->pinned_free.emplace_back(b.h_tot, b.h_bytes);
    if (!failed) {
      // a window may still have been refused for its size, which the expectation cannot have foreseen: keep what the plan found
      for (u32 k = 0; k < b.n; ++k) {
        auto it = ctx->windows.find(b.first + k);
        if (it != ctx->windows.end() && it->second.analysed) std::memcpy(it->second.totals, b.h_tot + (size_t)k * T_COUNT, sizeof it->second.totals);
      }
      continue;
    }
  }
  if (!failed) return CCLD_OK;
  CK(cudaMemsetAsync(ctx->d_poison, 0, 4, ctx->stream));
  failed = false;
  for (PendingBatch& b : todo) {
    if (!failed) { for (u32 k = 0; k < b.n && !failed; ++k) if (b.h_tot[(size_t)k * T_COUNT + T_FAILED] == FAILED_EXPECT) failed = true; }
    if (!failed) continue;
    bool present = true;
    for (u32 k = 0; k < b.n; ++k) {
      auto it = ctx->windows.find(b.first + k);
      if (it == ctx->windows.end()) { present = false; continue; }
      drop_results(it->second);
    }
    if (!present) continue;                                // released in the meantime: nothing to analyse
    const int r = analyze_batch(ctx, b.first, b.n, b.now, false);
    if (r != CCLD_OK && rc == CCLD_OK) rc = r;
  }
  return rc;
}

int find_analysed(ccld_ctx* ctx, u32 wid, WindowHost** out) {
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  auto it = ctx->windows.find(wid);
  if (it == ctx->windows.end()) return fail(ctx, CCLD_ERR_NO_WINDOW, "unknown window id");
  if (!it->second.analysed) return fail(ctx, CCLD_ERR_NO_WINDOW, "window not analysed");
  *out = &it->second;
  return CCLD_OK;
}

}  // namespace

extern "C" {

void ccld_params_default(ccld_params* p) {
  if (!p) return;
  p->tbase_init_ns = 2000000; p->theta_slow_milli = 3000; p->alpha_milli = 400; p->beta_milli = 600;
  p->m_max_rounds = 100; p->m_max_ns = 120000000000ll; p->hang_ns = 300000000000ll; p->barrier_bytes = 4;
  p->slow_rep_threshold = 1; p->k_milli = 5189; p->min_group = 4; p->vote_rep_milli = 100;
}

int ccld_create(ccld_ctx** out, const ccld_params* params, int device, void* cuda_stream) {
  if (!out || !params) return CCLD_ERR_ARG;
  *out = nullptr;
  if (params->tbase_init_ns <= 0 || params->m_max_rounds == 0 || params->m_max_ns <= 0 || params->min_group == 0) return CCLD_ERR_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return CCLD_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return CCLD_ERR_CUDA;
  ccld_ctx* ctx = new (std::nothrow) ccld_ctx();
  if (!ctx) return CCLD_ERR_NOMEM;
  ctx->params = *params; ctx->device = device; ctx->stream = (cudaStream_t)cuda_stream;
  { int sms = 0; if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess && sms > 0) ctx->n_sms = (u32)sms; }
  Params& d = ctx->dp;
  d.tbase_init_ns = params->tbase_init_ns; d.m_max_ns = params->m_max_ns; d.hang_ns = params->hang_ns; d.barrier_bytes = params->barrier_bytes;
  d.theta_slow_milli = params->theta_slow_milli; d.alpha_milli = params->alpha_milli; d.beta_milli = params->beta_milli;
  d.m_max_rounds = params->m_max_rounds; d.slow_rep_threshold = params->slow_rep_threshold; d.k_milli = params->k_milli;
  d.min_group = params->min_group; d.vote_rep_milli = params->vote_rep_milli;
  *out = ctx;
  return CCLD_OK;
}

int ccld_destroy(ccld_ctx* ctx) {
  if (!ctx) return CCLD_ERR_ARG;
  cudaSetDevice(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  for (auto& kv : ctx->windows) { drop_results(kv.second); if (kv.second.owns) ctx->pool.put(kv.second.own); }
  ctx->windows.clear();
  ctx->pool.put(ctx->reg_blk); ctx->pool.put(ctx->misc_blk);
  ctx->pool.clear();
  if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
  for (auto& b : ctx->pending) cudaFreeHost(b.h_tot);
  for (auto& f : ctx->pinned_free) cudaFreeHost(f.first);
  for (auto& sl : ctx->ring) for (int i = 0; i < TIMER_PAIRS; ++i) { cudaEventDestroy(sl.a[i]); cudaEventDestroy(sl.b[i]); }
  delete ctx;
  return CCLD_OK;
}

const char* ccld_last_error(ccld_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int ccld_comm_register(ccld_ctx* ctx, uint32_t comm, const uint32_t* ranks, uint32_t n, uint8_t algo, uint32_t seq0) {
  if (!ctx) return CCLD_ERR_ARG;
  if (ctx->finalized) return fail(ctx, CCLD_ERR_STATE, "communicators must be registered before the first analysis");
  if (!ranks || n == 0) return fail(ctx, CCLD_ERR_ARG, "empty communicator");
  if (algo > 1) return fail(ctx, CCLD_ERR_ARG, "algo must be 0 (ring) or 1 (tree)");
  if (n > CCLD_MAX_COMM_SIZE) return fail(ctx, CCLD_ERR_CAPACITY, "communicator larger than CCLD_MAX_COMM_SIZE");
  if (ctx->comm_idx.count(comm)) return fail(ctx, CCLD_ERR_ARG, "communicator id registered twice");
  CommHost c; c.id = comm; c.seq0 = seq0; c.algo = algo; c.ranks.assign(ranks, ranks + n);
  std::vector<u32> sorted(c.ranks); std::sort(sorted.begin(), sorted.end());
  if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return fail(ctx, CCLD_ERR_ARG, "rank listed twice in a communicator");
  if (sorted.back() >= CCLD_MAX_RANK_ID) return fail(ctx, CCLD_ERR_CAPACITY, "rank id not below CCLD_MAX_RANK_ID");
  ctx->comm_idx[comm] = (u32)ctx->comms.size();
  ctx->comms.push_back(std::move(c));
  return CCLD_OK;
}

int ccld_comm_set_layers(ccld_ctx* ctx, uint32_t comm, const uint32_t* layer) {
  if (!ctx) return CCLD_ERR_ARG;
  if (ctx->finalized) return fail(ctx, CCLD_ERR_STATE, "layers must be set before the first analysis");
  if (!layer) return fail(ctx, CCLD_ERR_ARG, "layer is null");
  auto ci = ctx->comm_idx.find(comm);
  if (ci == ctx->comm_idx.end()) return fail(ctx, CCLD_ERR_UNKNOWN_COMM, "unknown communicator");
  CommHost& c = ctx->comms[ci->second];
  if (c.algo != 1) return fail(ctx, CCLD_ERR_ARG, "layers belong to tree communicators (algo 1)");
  const u32 n = (u32)c.ranks.size();
  std::unordered_map<u32, u32> first;       // layer id -> lowest position that carries it
  c.head.resize(n);
  for (u32 p = 0; p < n; ++p) c.head[p] = first.emplace(layer[p], p).first->second;
  return CCLD_OK;
}

int ccld_trace_upload(ccld_ctx* ctx, uint32_t window_id, uint64_t n_rec, int mem_kind,
                      const uint32_t* rank, const uint32_t* comm, const uint32_t* seq, const uint8_t* op,
                      const uint64_t* bytes, const int64_t* t_enter_ns, const int64_t* t_exit_ns,
                      const uint32_t* send_chg, const uint32_t* recv_chg,
                      uint32_t n_frames, const uint32_t* f_rank, const uint32_t* f_comm, const uint32_t* f_seq,
                      uint32_t n_channels, const uint32_t* progress) {
  NvtxRange nvtx_range("ccld_trace_upload");
  if (!ctx) return CCLD_ERR_ARG;
  if (mem_kind != 0 && mem_kind != 1) return fail(ctx, CCLD_ERR_ARG, "mem_kind must be 0 (host) or 1 (device)");
  if (n_rec >= 0xFFFFFFFFull) return fail(ctx, CCLD_ERR_CAPACITY, "window of 2^32 - 1 or more records");
  if (n_rec > 0 && (!rank || !comm || !seq || !op || !bytes || !t_enter_ns || !t_exit_ns)) return fail(ctx, CCLD_ERR_ARG, "null column");
  if ((send_chg == nullptr) != (recv_chg == nullptr)) return fail(ctx, CCLD_ERR_ARG, "send_chg and recv_chg must both be given or both be null");
  if (n_frames > 0 && (!f_rank || !f_comm || !f_seq || !progress || n_channels == 0)) return fail(ctx, CCLD_ERR_ARG, "incomplete progress frames");
  if (ctx->windows.count(window_id)) return fail(ctx, CCLD_ERR_STATE, "window id already uploaded");
  CK(cudaSetDevice(ctx->device));
  WindowHost w; w.id = window_id; w.n_rec = n_rec; w.n_frames = n_frames; w.n_channels = n_channels;
  WinDesc& d = w.d;
  d.n_rec = n_rec;
  if (mem_kind == 1) {
    d.rank = rank; d.comm = comm; d.seq = seq; d.op = op; d.bytes = bytes; d.t_enter = t_enter_ns; d.t_exit = t_exit_ns;
    d.send_chg = send_chg; d.recv_chg = recv_chg;
    w.f_rank = f_rank; w.f_comm = f_comm; w.f_seq = f_seq; w.progress = progress;
  } else {
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off = align_up(off + b); return o; };
    const size_t o_rank = take(n_rec * 4), o_comm = take(n_rec * 4), o_seq = take(n_rec * 4), o_op = take(n_rec), o_bytes = take(n_rec * 8),
                 o_te = take(n_rec * 8), o_tx = take(n_rec * 8), o_sc = take(send_chg ? n_rec * 4 : 0), o_rc = take(recv_chg ? n_rec * 4 : 0),
                 o_fr = take(n_frames * 4ull), o_fc = take(n_frames * 4ull), o_fs = take(n_frames * 4ull), o_pr = take((size_t)n_frames * n_channels * 8);
    cudaError_t e;
    w.own = ctx->pool.get(off, &e);
    if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "window allocation failed");
    w.owns = true;
    char* b = (char*)w.own.p; cudaStream_t st = ctx->stream;
    auto up = [&](size_t o, const void* src, size_t nb) { return nb ? cudaMemcpyAsync(b + o, src, nb, cudaMemcpyHostToDevice, st) : cudaSuccess; };
    cudaError_t ce = cudaSuccess;
    auto acc = [&](cudaError_t x) { if (ce == cudaSuccess) ce = x; };
    acc(up(o_rank, rank, n_rec * 4)); acc(up(o_comm, comm, n_rec * 4)); acc(up(o_seq, seq, n_rec * 4)); acc(up(o_op, op, n_rec));
    acc(up(o_bytes, bytes, n_rec * 8)); acc(up(o_te, t_enter_ns, n_rec * 8)); acc(up(o_tx, t_exit_ns, n_rec * 8));
    if (send_chg) { acc(up(o_sc, send_chg, n_rec * 4)); acc(up(o_rc, recv_chg, n_rec * 4)); }
    if (n_frames) { acc(up(o_fr, f_rank, n_frames * 4ull)); acc(up(o_fc, f_comm, n_frames * 4ull)); acc(up(o_fs, f_seq, n_frames * 4ull));
                    acc(up(o_pr, progress, (size_t)n_frames * n_channels * 8)); }
    if (ce != cudaSuccess) { ctx->pool.put(w.own); return fail(ctx, CCLD_ERR_CUDA, std::string("upload copy: ") + cudaGetErrorString(ce)); }
    d.rank = (const u32*)(b + o_rank); d.comm = (const u32*)(b + o_comm); d.seq = (const u32*)(b + o_seq); d.op = (const u8*)(b + o_op);
    d.bytes = (const u64*)(b + o_bytes); d.t_enter = (const i64*)(b + o_te); d.t_exit = (const i64*)(b + o_tx);
    d.send_chg = send_chg ? (const u32*)(b + o_sc) : nullptr; d.recv_chg = recv_chg ? (const u32*)(b + o_rc) : nullptr;
    if (n_frames) { w.f_rank = (const u32*)(b + o_fr); w.f_comm = (const u32*)(b + o_fc); w.f_seq = (const u32*)(b + o_fs); w.progress = (const u32*)(b + o_pr); }
  }
  ctx->windows.emplace(window_id, std::move(w));
  return CCLD_OK;
}

int ccld_window_release(ccld_ctx* ctx, uint32_t window_id) {
  if (!ctx) return CCLD_ERR_ARG;
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  auto it = ctx->windows.find(window_id);
  if (it == ctx->windows.end()) return fail(ctx, CCLD_ERR_NO_WINDOW, "unknown window id");
  CK(cudaSetDevice(ctx->device));
  CK(cudaStreamSynchronize(ctx->stream));     // nothing in flight may still read the blocks we recycle
  drop_results(it->second);
  if (it->second.owns) ctx->pool.put(it->second.own);
  if (it->second.owns_opset) ctx->pool.put(it->second.opset_own);
  ctx->windows.erase(it);
  return CCLD_OK;
}

int ccld_reset(ccld_ctx* ctx) {
  if (!ctx) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  CK(cudaStreamSynchronize(ctx->stream));
  // batches still in doubt need no second analysis: their results are dropped with all the others
  for (auto& b : ctx->pending) ctx->pinned_free.emplace_back(b.h_tot, b.h_bytes);
  ctx->pending.clear();
  for (auto& kv : ctx->windows) drop_results(kv.second);
  if (ctx->finalized) {
    CK(cudaMemsetAsync((char*)ctx->reg_blk.p + ctx->stats_off, 0, ctx->stats_bytes, ctx->stream));
    CK(cudaMemsetAsync(ctx->d_poison, 0, 4, ctx->stream));
  }
  return CCLD_OK;
}

int ccld_analyze_window(ccld_ctx* ctx, uint32_t first_window, uint32_t n_windows, int64_t now_ns) {
  NvtxRange nvtx_range("ccld_analyze_window");
  if (!ctx) return CCLD_ERR_ARG;
  if (n_windows == 0) return fail(ctx, CCLD_ERR_ARG, "n_windows is zero");
  if (n_windows > 65535) return fail(ctx, CCLD_ERR_CAPACITY, "more than 65,535 windows in one batch");
  return analyze_batch(ctx, first_window, n_windows, now_ns, ctx->speculate != 0);
}

int ccld_set_speculation(ccld_ctx* ctx, int on) {
  if (!ctx) return CCLD_ERR_ARG;
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  ctx->speculate = on != 0;
  return CCLD_OK;
}

}  // extern "C"

namespace {

int analyze_batch(ccld_ctx* ctx, u32 first_window, u32 n_windows, i64 now_ns, bool may_speculate) {
  CK(cudaSetDevice(ctx->device));
  std::vector<WindowHost*> ws(n_windows);
  for (u32 k = 0; k < n_windows; ++k) {
    auto it = ctx->windows.find(first_window + k);
    if (it == ctx->windows.end()) return fail(ctx, CCLD_ERR_NO_WINDOW, "window not uploaded");
    if (it->second.analysed) return fail(ctx, CCLD_ERR_STATE, "window already analysed");
    ws[k] = &it->second;
  }
  { int rc = finalize_registry(ctx); if (rc != CCLD_OK) return rc; }
  const u32 B = n_windows, nc = ctx->reg.n_comms;
  cudaStream_t st = ctx->stream;

  // A batch of a shape seen before (the same record count in every window) is enqueued without waiting for its plan:
  // the results are sized from the totals that shape had last time, and the plan checks them on the device.
  const ShapeEntry* expect = nullptr;
  if (may_speculate) {
    for (const ShapeEntry& e : ctx->shapes) {
      if (e.n_rec.size() != B) continue;
      bool same = true;
      for (u32 k = 0; k < B && same; ++k) same = e.n_rec[k] == ws[k]->n_rec;
      if (same) { expect = &e; break; }
    }
  }
  if (!expect) { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }    // the waiting path runs with nothing in doubt before it

  // ---- plan block: descriptors, op-counter ranges, layout rows, totals, counters ----
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up(off + b); return o; };
  const size_t o_desc = take(B * sizeof(WinDesc)), o_rmin = take((size_t)B * nc * 4), o_rmax = take((size_t)B * nc * 4),
               o_rng = take((size_t)B * nc * sizeof(RangeRow)), o_srow = take((size_t)B * nc * sizeof(uint4)), o_rent = take((size_t)B * ctx->n_ranks * RANK_TAB_K * sizeof(uint4)), o_tot = take((size_t)B * T_COUNT * 8), o_cnt = take((size_t)B * C_COUNT * 8),
               o_zero_end = off, o_exp = take(expect ? (size_t)B * T_COUNT * 8 : 0);
  cudaError_t e;
  Block pb = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "plan allocation failed");
  auto plan_blk = std::make_shared<Shared>(&ctx->pool, pb);
  char* pbase = (char*)pb.p;
  std::vector<WinDesc> hd(B);
  u64 cta = 0;
  for (u32 k = 0; k < B; ++k) {
    WinDesc d = ws[k]->d;
    d.slot_cap = 2 * d.n_rec + ctx->sum_n;
    d.n_cta = (u32)((d.n_rec + REC_PER_CTA - 1) / REC_PER_CTA); d.cta0 = 0; cta = std::max<u64>(cta, d.n_cta);
    d.rmin = (u32*)(pbase + o_rmin) + (size_t)k * nc; d.rmax = (u32*)(pbase + o_rmax) + (size_t)k * nc;
    d.ranges = (RangeRow*)(pbase + o_rng) + (size_t)k * nc; d.srow = (uint4*)(pbase + o_srow) + (size_t)k * nc;
    d.rent = (uint4*)(pbase + o_rent) + (size_t)k * ctx->n_ranks * RANK_TAB_K;
    d.totals = (u64*)(pbase + o_tot) + (size_t)k * T_COUNT; d.counters = (u64*)(pbase + o_cnt) + (size_t)k * C_COUNT;
    d.expect = expect ? (const u64*)(pbase + o_exp) + (size_t)k * T_COUNT : nullptr; d.poison = ctx->d_poison;
    d.n_groups = d.n_slots = 0; d.perm = nullptr; d.flags = nullptr; d.skey = d.dkey = nullptr; d.gi64 = nullptr; d.gu32 = nullptr; d.gbw = nullptr;
    d.comm_rows = nullptr; d.alerts = nullptr;
    for (int q = 0; q < B_COUNT; ++q) d.base[q] = 0;
    d.pad = 0; d.tsum[0] = d.tsum[1] = d.tsum[2] = nullptr;
    hd[k] = d;
  }
  if (cta > 0x7FFFFFFFull) return fail(ctx, CCLD_ERR_CAPACITY, "batch too large for one launch");
  WinDesc* d_desc = (WinDesc*)(pbase + o_desc);
  TimerSlot* ts = timer_begin(ctx);
  auto start_plan = [&]() -> cudaError_t {               // clears the plan block, uploads the descriptors, runs the range pass and the layout
    cudaError_t r = cudaMemsetAsync(pbase, 0, o_zero_end, st);
    if (r == cudaSuccess) r = cudaMemsetAsync(pbase + o_rmin, 0xFF, (size_t)B * nc * 4, st);
    if (r == cudaSuccess && expect) r = cudaMemcpyAsync(pbase + o_exp, expect->totals.data(), (size_t)B * T_COUNT * 8, cudaMemcpyHostToDevice, st);
    if (r == cudaSuccess) r = cudaMemcpyAsync(d_desc, hd.data(), B * sizeof(WinDesc), cudaMemcpyHostToDevice, st);
    if (r != cudaSuccess) return r;
    if (cta > 0) {
      // enough CTAs to fill the device several times over, then as many blocks per CTA as that leaves
      const u64 want = 32ull * ctx->n_sms;
      const u32 per = (u32)std::min<u64>(RANGE_BLOCKS_MAX, std::max<u64>(1, cta * B / want));
      TimedLaunch tl(ts, 0, st);
      k_seq_range<<<dim3((u32)((cta + per - 1) / per), B), REC_THREADS, range_smem_bytes(nc), st>>>(d_desc, ctx->reg, per);
    }
    { TimedLaunch tl(ts, 1, st); k_plan<<<B, PLAN_THREADS, 0, st>>>(d_desc, ctx->reg, PlanLists{nullptr, nullptr, nullptr, nullptr}, 0); }
    return cudaGetLastError();
  };
  const u64* tot = nullptr;                                // [B][T_COUNT] totals the results are sized from
  if (!expect) {
    CK(start_plan());
    { int rc = ensure_pinned(ctx, (size_t)B * T_COUNT * 8); if (rc != CCLD_OK) return rc; }
    CK(cudaMemcpyAsync(ctx->h_pinned, pbase + o_tot, (size_t)B * T_COUNT * 8, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    tot = ctx->h_pinned;
  } else tot = expect->totals.data();

  // ---- result block: sized from the totals ----
  off = 0;
  u64 total_slots = 0, n_list[B_COUNT] = {0, 0, 0, 0, 0};       // batch-wide list lengths (B_*)
  const int t_of[B_COUNT] = {T_FCTA, T_FWT, T_FSUM, T_TILES2, T_TILES3};
  for (u32 k = 0; k < B; ++k) { const u64* t = tot + (size_t)k * T_COUNT; total_slots += t[T_SLOTS]; }
  const size_t o_perm = take(total_slots * 4 + ALIGN);
  std::vector<size_t> o_flags(B), o_gi(B), o_gu(B), o_gb(B), o_rows(B), o_al(B), perm_off(B);
  { size_t po = 0;
    for (u32 k = 0; k < B; ++k) {
      const u64* t = tot + (size_t)k * T_COUNT;
      perm_off[k] = po; po += t[T_SLOTS] * 4;
      o_flags[k] = take(t[T_SLOTS]); o_gi[k] = take(t[T_GROUPS] * 8 * GI_COUNT); o_gu[k] = take(t[T_GROUPS] * 4 * GU_COUNT);
      o_gb[k] = take(t[T_GROUPS] * 8); o_rows[k] = take(t[T_ROWS] * sizeof(ccld_comm_verdict));
      o_al[k] = take(CCLD_MAX_ALERTS_PER_WINDOW * sizeof(ccld_hang_alert));
      for (int q = 0; q < B_COUNT; ++q) { hd[k].base[q] = (u32)n_list[q]; n_list[q] += t[t_of[q]]; }
    } }
  for (int q = 0; q < B_COUNT; ++q) if (n_list[q] > 0x7FFFFFFFull) return fail(ctx, CCLD_ERR_CAPACITY, "too many tiles in one batch");
  const size_t o_fcta = take(n_list[B_FCTA] * sizeof(FusedCta)), o_fwt = take(n_list[B_FWT] * sizeof(WarpTile)),
               o_fsum = take(n_list[B_FSUM] * sizeof(TileSum)), o_t2 = take(n_list[B_T2] * sizeof(Tile)), o_s2 = take(n_list[B_T2] * sizeof(TileSum)),
               o_t3 = take(n_list[B_T3] * sizeof(Tile)), o_s3 = take(n_list[B_T3] * sizeof(TileSum));
  // groups the fused kernel may set aside for the deferred kernel: at most every group of the batch
  u64 total_groups = 0;
  for (u32 k = 0; k < B; ++k) total_groups += tot[(size_t)k * T_COUNT + T_GROUPS];
  const size_t o_defn = take(16), o_def = take(n_list[B_FCTA] ? total_groups * 8 : 0),
               o_def3 = take(n_list[B_T3] * (size_t)LARGE_SEQS * 8),          // likewise for the kernel of the largest communicators
               o_lgrp = take(n_list[B_T3] * (size_t)LARGE_SEQS * sizeof(LargeGroup)),
               o_skey = take(n_list[B_T3] ? total_slots * 4 : 0), o_dkey = take(n_list[B_T3] ? total_slots * 4 : 0);
  Block rb = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "result allocation failed");
  auto res_blk = std::make_shared<Shared>(&ctx->pool, rb);
  char* rbase = (char*)rb.p;
  for (u32 k = 0; k < B; ++k) {
    const u64* t = tot + (size_t)k * T_COUNT;
    WinDesc& d = hd[k];
    d.n_groups = t[T_GROUPS]; d.n_slots = t[T_SLOTS];
    d.perm = (u32*)(rbase + o_perm + perm_off[k]); d.flags = (u8*)(rbase + o_flags[k]);
    if (n_list[B_T3]) { d.skey = (u32*)(rbase + o_skey + perm_off[k]); d.dkey = (u32*)(rbase + o_dkey + perm_off[k]); }
    d.gi64 = (i64*)(rbase + o_gi[k]); d.gu32 = (u32*)(rbase + o_gu[k]); d.gbw = (double*)(rbase + o_gb[k]);
    d.comm_rows = (ccld_comm_verdict*)(rbase + o_rows[k]); d.alerts = (ccld_hang_alert*)(rbase + o_al[k]);
    d.tsum[0] = (TileSum*)(rbase + o_fsum); d.tsum[1] = (TileSum*)(rbase + o_s2); d.tsum[2] = (TileSum*)(rbase + o_s3);
  }
  if (expect) CK(start_plan());                            // descriptors already complete: nothing was waited for
  else CK(cudaMemcpyAsync(d_desc, hd.data(), B * sizeof(WinDesc), cudaMemcpyHostToDevice, st));
  if (total_slots) CK(cudaMemsetAsync(rbase + o_perm, 0xFF, total_slots * 4, st));
  PlanLists pl; pl.fcta = (FusedCta*)(rbase + o_fcta); pl.fwt = (WarpTile*)(rbase + o_fwt); pl.t2 = (Tile*)(rbase + o_t2); pl.t3 = (Tile*)(rbase + o_t3);
  { TimedLaunch tl(ts, 1, st); k_plan<<<B, PLAN_THREADS, 0, st>>>(d_desc, ctx->reg, pl, 1); }
  if (cta > 0) {
    const u64 blocks = (cta * REC_PER_CTA + SCAT_PER_CTA - 1) / SCAT_PER_CTA;      // of the largest window
    const u32 per = (u32)std::min<u64>(SCAT_BLOCKS_MAX, std::max<u64>(1, blocks * B / (16ull * ctx->n_sms)));
    TimedLaunch tl(ts, 2, st);
    k_slot_scatter<<<dim3((u32)((blocks + per - 1) / per), B), SCAT_THREADS, 0, st>>>(d_desc, ctx->reg, per);
  }
  CK(cudaMemsetAsync(rbase + o_defn, 0, 16, st));
  if (n_list[B_FCTA]) {
    const DeferList dl{(u64*)(rbase + o_def), (u32*)(rbase + o_defn)};
    TimedLaunch tl(ts, 3, st);
    k_reduce_fused<<<(u32)n_list[B_FCTA], SMALL_SEQS, 0, st>>>(d_desc, pl.fcta, pl.fwt, (TileSum*)(rbase + o_fsum), ctx->reg, ctx->dp, dl);
    k_reduce_deferred<<<DEF_GRID, DEF_WARPS * 32, 0, st>>>(d_desc, dl, ctx->reg, ctx->dp, now_ns);
  }
  if (n_list[B_T2]) { TimedLaunch tl(ts, 4, st); k_reduce_mid<<<(u32)n_list[B_T2], MID_THREADS, mid_smem_bytes(2 * WARP_N), st>>>(d_desc, pl.t2, (TileSum*)(rbase + o_s2), ctx->reg, ctx->dp, now_ns); }
  if (n_list[B_T3]) {
    const DeferList dl{(u64*)(rbase + o_def3), (u32*)(rbase + o_defn) + 2};
    LargeGroup* lgrp = (LargeGroup*)(rbase + o_lgrp);
    CK(cudaMemsetAsync(lgrp, 0, n_list[B_T3] * (size_t)LARGE_SEQS * sizeof(LargeGroup), st));
    TimedLaunch tl(ts, 5, st);
    k_large_stage<<<dim3((u32)n_list[B_T3], (ctx->max_large_n + LS_MEMBERS - 1) / LS_MEMBERS), LS_THREADS, 0, st>>>(d_desc, pl.t3, lgrp, ctx->reg);
    const u32 grid = (u32)std::min<u64>(n_list[B_T3], 2ull * ctx->n_sms);      // persistent: two CTAs per SM take the tiles in turn
    k_reduce_large<<<grid, LG_THREADS, ctx->large_smem, st>>>(d_desc, pl.t3, (u32)n_list[B_T3], lgrp, (TileSum*)(rbase + o_s3), ctx->reg, ctx->dp, dl);
    k_reduce_large_deferred<<<LARGE_DEF_GRID, LARGE_DEF_THREADS, 16ull * ctx->max_large_n, st>>>(d_desc, dl, ctx->reg, ctx->dp, now_ns);
  }
  {
    TimedLaunch tl(ts, 6, st);
    k_window_rounds<<<dim3((nc + 3) / 4, B), 128, 0, st>>>(d_desc, ctx->reg);
    k_window_decide<<<(nc + 3) / 4, 128, 0, st>>>(d_desc, B, ctx->reg, ctx->dp);
    if (ctx->n_trees) k_tree_root_comm<<<dim3(ctx->n_trees, B), TREE_THREADS, 0, st>>>(d_desc, ctx->d_trees, ctx->reg);
  }
  CK(cudaGetLastError());
  for (u32 k = 0; k < B; ++k) {
    WindowHost& w = *ws[k];
    w.analysed = true; w.plan_blk = plan_blk; w.res_blk = res_blk; w.d_desc = d_desc + k; w.d = hd[k];
    std::memcpy(w.totals, tot + (size_t)k * T_COUNT, sizeof w.totals);
  }
  if (expect) {
    // what the plan really found follows the batch into pinned memory; settle() reads it
    PendingBatch pbatch; pbatch.first = first_window; pbatch.n = B; pbatch.now = now_ns;
    pbatch.h_tot = pinned_get(ctx, (size_t)B * T_COUNT * 8, &pbatch.h_bytes);
    if (!pbatch.h_tot) { cudaStreamSynchronize(st); return fail(ctx, CCLD_ERR_NOMEM, "pinned allocation failed"); }
    CK(cudaMemcpyAsync(pbatch.h_tot, pbase + o_tot, (size_t)B * T_COUNT * 8, cudaMemcpyDeviceToHost, st));
    ctx->pending.push_back(pbatch);
  } else {
    // remember the totals of this shape, unless a window was refused
    bool clean = true;
    for (u32 k = 0; k < B && clean; ++k) clean = tot[(size_t)k * T_COUNT + T_FAILED] == 0;
    if (clean) {
      ShapeEntry se; se.n_rec.resize(B); se.totals.assign(tot, tot + (size_t)B * T_COUNT);
      for (u32 k = 0; k < B; ++k) se.n_rec[k] = ws[k]->n_rec;
      for (size_t i = 0; i < ctx->shapes.size(); ++i) if (ctx->shapes[i].n_rec == se.n_rec) { ctx->shapes.erase(ctx->shapes.begin() + i); break; }
      if (ctx->shapes.size() >= SHAPE_CACHE) ctx->shapes.erase(ctx->shapes.begin());
      ctx->shapes.push_back(std::move(se));
    }
  }
  return CCLD_OK;
}

}  // namespace

extern "C" {

int ccld_get_verdict(ccld_ctx* ctx, uint32_t window_id, ccld_verdict* out) {
  NvtxRange nvtx_range("ccld_get_verdict");
  if (!ctx || !out) return CCLD_ERR_ARG;
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->stream;
  u64 cnt[C_COUNT];
  CK(cudaMemcpyAsync(cnt, w->d.counters, sizeof cnt, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  out->n_records = w->n_rec; out->n_groups = w->totals[T_GROUPS]; out->n_slots = w->totals[T_SLOTS];
  out->n_rejected = w->n_rec - cnt[C_PRESENT]; out->n_complete = cnt[C_COMPLETE]; out->n_incomplete = cnt[C_INCOMPLETE];
  out->n_barrier = cnt[C_BARRIER]; out->n_analysed = cnt[C_ANALYSED]; out->n_flag_skew = cnt[C_FLAG_SKEW]; out->n_flag_dur = cnt[C_FLAG_DUR];
  out->n_opset_mismatch = cnt[C_MISMATCH];
  u32 err = (u32)cnt[C_ERR];
  if (!w->totals[T_FAILED] && w->n_rec - cnt[C_PRESENT] != cnt[C_REJECTED]) err |= CCLD_E_DUPLICATE;   // a slot was written twice
  out->error_bits = err;
  out->n_comm_rows_total = (u32)w->totals[T_ROWS];
  const u32 n_rows = std::min<u32>(out->n_comm_rows_total, out->comm_rows ? out->comm_rows_cap : 0);
  if (n_rows) CK(cudaMemcpyAsync(out->comm_rows, w->d.comm_rows, n_rows * sizeof(ccld_comm_verdict), cudaMemcpyDeviceToHost, st));
  char* m = (char*)ctx->misc_blk.p;
  const MiscLayout L = misc_layout(ctx->n_ranks, ctx->max_n);
  ccld_suspect* sus_a = (ccld_suspect*)(m + L.sus_a); ccld_suspect* sus_b = (ccld_suspect*)(m + L.sus_b);
  ccld_hang_alert* al_b = (ccld_hang_alert*)(m + L.alerts);
  u32* d_count = (u32*)(m + L.count);
  // hang alerts, ordered by (communicator, seq)
  out->n_alerts_total = (u32)std::min<u64>(cnt[C_ALERTS], 0xFFFFFFFFull);
  const u32 n_al_dev = std::min<u32>(out->n_alerts_total, CCLD_MAX_ALERTS_PER_WINDOW);
  const u32 n_al = std::min<u32>(n_al_dev, out->alerts ? out->alerts_cap : 0);
  if (n_al) {
    k_rank_sort_alerts<<<(n_al_dev + 127) / 128, 128, 0, st>>>(w->d.alerts, n_al_dev, al_b, ctx->reg);
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(out->alerts, al_b, n_al * sizeof(ccld_hang_alert), cudaMemcpyDeviceToHost, st));
  }
  // cumulative suspects
  const u32 sus_cap = 2 * ctx->n_ranks;
  u32 n_sus = 0;
  CK(cudaMemsetAsync(d_count, 0, 4, st));
  k_suspects<<<(ctx->n_ranks + 255) / 256, 256, 0, st>>>(ctx->reg, ctx->dp, sus_a, sus_cap, d_count);
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(&n_sus, d_count, 4, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  out->n_suspects_total = n_sus;
  const u32 n_out = std::min<u32>(n_sus, out->suspects ? out->suspects_cap : 0);
  if (n_out) {
    k_rank_sort_suspects<<<(n_sus + 127) / 128, 128, 0, st>>>(sus_a, n_sus, sus_b);
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(out->suspects, sus_b, n_out * sizeof(ccld_suspect), cudaMemcpyDeviceToHost, st));
  }
  CK(cudaStreamSynchronize(st));
  if (cnt[C_INTERNAL]) return fail(ctx, CCLD_ERR_CUDA, "internal: slot index out of range");
  if (err & CCLD_E_UNKNOWN_COMM) return fail(ctx, CCLD_ERR_UNKNOWN_COMM, "record of an unregistered communicator");
  if (err & CCLD_E_NOT_MEMBER) return fail(ctx, CCLD_ERR_NOT_MEMBER, "record of a rank that is not a member of its communicator");
  if (err & CCLD_E_SEQ_RANGE) return fail(ctx, CCLD_ERR_SEQ_RANGE, "record with an op counter below the communicator's first");
  if (err & CCLD_E_DUPLICATE) return fail(ctx, CCLD_ERR_DUPLICATE, "duplicate (communicator, op counter, rank) record");
  if (err & CCLD_E_CAPACITY) return fail(ctx, CCLD_ERR_CAPACITY, "op counters of the window span too many slots");
  return CCLD_OK;
}

// Tree communicators compare progress counters inside a layer; the kernel needs the layer table for that.
static int hang_layers(ccld_ctx* ctx, const CommHost& c, HangArgs* A) {
  A->head = nullptr;
  if (c.algo == 0) return CCLD_OK;
  if (!c.d_head) return fail(ctx, CCLD_ERR_STATE, "tree communicator without layers (ccld_comm_set_layers)");
  A->head = c.d_head;
  return CCLD_OK;
}

int ccld_locate_hang(ccld_ctx* ctx, uint32_t window_id, uint32_t comm, uint32_t seq, ccld_hang_verdict* out) {
  NvtxRange nvtx_range("ccld_locate_hang");
  if (!ctx || !out) return CCLD_ERR_ARG;
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  auto ci = ctx->comm_idx.find(comm);
  if (ci == ctx->comm_idx.end()) return fail(ctx, CCLD_ERR_UNKNOWN_COMM, "unknown communicator");
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->stream;
  const u32 n = (u32)ctx->comms[ci->second].ranks.size();
  char* m = (char*)ctx->misc_blk.p;
  const MiscLayout L = misc_layout(ctx->n_ranks, ctx->max_n);
  HangArgs A;
  A.c = ci->second; A.seq = seq; A.n_frames = w->n_frames; A.n_channels = w->n_channels;
  A.f_rank = w->f_rank; A.f_comm = w->f_comm; A.f_seq = w->f_seq; A.progress = w->progress;
  A.entered = (u8*)(m + L.entered); A.done = (u8*)(m + L.done); A.frame = (u32*)(m + L.frame); A.roots = (u32*)(m + L.roots);
  A.tot = (u64*)(m + L.tot); A.out = (ccld_hang_verdict*)(m + L.hang_out);
  A.roots_cap = n;
  { int rc = hang_layers(ctx, ctx->comms[ci->second], &A); if (rc != CCLD_OK) return rc; }
  k_hang_locate<<<1, 1024, 0, st>>>(w->d_desc, ctx->reg, A);
  CK(cudaGetLastError());
  ccld_hang_verdict v;
  CK(cudaMemcpyAsync(&v, A.out, sizeof v, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  u32* roots = out->roots; const u32 cap = roots ? out->roots_cap : 0;
  *out = v; out->roots = roots; out->roots_cap = cap;
  const u32 n_copy = std::min<u32>(std::min<u32>(v.n_roots_total, n), cap);
  if (n_copy) { CK(cudaMemcpyAsync(roots, A.roots, n_copy * 4ull, cudaMemcpyDeviceToHost, st)); CK(cudaStreamSynchronize(st)); }
  return CCLD_OK;
}

int ccld_locate_hangs(ccld_ctx* ctx, uint32_t window_id, ccld_hang_alert* alerts, ccld_hang_verdict* out, uint32_t cap,
                      uint32_t* roots, uint32_t roots_stride, uint32_t* n_total) {
  if (!ctx || !n_total) return CCLD_ERR_ARG;
  if (cap && !out) return fail(ctx, CCLD_ERR_ARG, "out is null");
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->stream;
  u64 n_al64 = 0;
  CK(cudaMemcpyAsync(&n_al64, w->d.counters + C_ALERTS, 8, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  *n_total = (u32)std::min<u64>(n_al64, 0xFFFFFFFFull);
  const u32 n_dev = (u32)std::min<u64>(n_al64, CCLD_MAX_ALERTS_PER_WINDOW), n = std::min<u32>(n_dev, cap);
  if (n == 0) return CCLD_OK;
  // the alerts in the order ccld_get_verdict lists them
  char* m = (char*)ctx->misc_blk.p;
  const MiscLayout L = misc_layout(ctx->n_ranks, ctx->max_n);
  ccld_hang_alert* al_b = (ccld_hang_alert*)(m + L.alerts);
  k_rank_sort_alerts<<<(n_dev + 127) / 128, 128, 0, st>>>(w->d.alerts, n_dev, al_b, ctx->reg);
  CK(cudaGetLastError());
  std::vector<ccld_hang_alert> al(n);
  CK(cudaMemcpyAsync(al.data(), al_b, n * sizeof(ccld_hang_alert), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  // per alert: scratch over the communicator's members, a root list and a verdict
  std::vector<HangArgs> ha(n);
  std::vector<size_t> o_roots(n);
  std::vector<u32> members(n);
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up(off + b); return o; };
  const size_t o_args = take(n * sizeof(HangArgs)), o_out = take(n * sizeof(ccld_hang_verdict));
  std::vector<size_t> o_ent(n), o_done(n), o_frame(n), o_tot(n);
  for (u32 i = 0; i < n; ++i) {
    auto ci = ctx->comm_idx.find(al[i].comm);
    if (ci == ctx->comm_idx.end()) return fail(ctx, CCLD_ERR_CUDA, "internal: alert names an unknown communicator");
    const u32 nm = (u32)ctx->comms[ci->second].ranks.size();
    members[i] = nm; ha[i].c = ci->second;
    { int rc = hang_layers(ctx, ctx->comms[ci->second], &ha[i]); if (rc != CCLD_OK) return rc; }
    o_ent[i] = take(nm); o_done[i] = take(nm); o_frame[i] = take(nm * 4ull); o_tot[i] = take(nm * 8ull); o_roots[i] = take(nm * 4ull);
  }
  cudaError_t e;
  Block blk = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "scratch allocation failed");
  char* b = (char*)blk.p;
  for (u32 i = 0; i < n; ++i) {
    HangArgs& A = ha[i];
    A.seq = al[i].seq; A.n_frames = w->n_frames; A.n_channels = w->n_channels;
    A.f_rank = w->f_rank; A.f_comm = w->f_comm; A.f_seq = w->f_seq; A.progress = w->progress;
    A.entered = (u8*)(b + o_ent[i]); A.done = (u8*)(b + o_done[i]); A.frame = (u32*)(b + o_frame[i]); A.tot = (u64*)(b + o_tot[i]);
    A.roots = (u32*)(b + o_roots[i]); A.roots_cap = members[i];
    A.out = (ccld_hang_verdict*)(b + o_out) + i;
  }
  std::vector<ccld_hang_verdict> hv(n);
  std::vector<char> host_blk;
  int rc = CCLD_OK;
  do {
    if (cudaMemcpyAsync(b + o_args, ha.data(), n * sizeof(HangArgs), cudaMemcpyHostToDevice, st) != cudaSuccess) { rc = CCLD_ERR_CUDA; break; }
    k_hang_locate_many<<<n, 1024, 0, st>>>(w->d_desc, ctx->reg, (const HangArgs*)(b + o_args));
    if (cudaGetLastError() != cudaSuccess) { rc = CCLD_ERR_CUDA; break; }
    host_blk.resize(off);
    // verdicts and root lists come back in one copy (they follow each other in the block)
    if (cudaMemcpyAsync(host_blk.data() + o_out, b + o_out, off - o_out, cudaMemcpyDeviceToHost, st) != cudaSuccess) { rc = CCLD_ERR_CUDA; break; }
    if (cudaStreamSynchronize(st) != cudaSuccess) { rc = CCLD_ERR_CUDA; break; }
  } while (0);
  ctx->pool.put(blk);
  if (rc != CCLD_OK) return fail(ctx, rc, "hang sweep failed");
  for (u32 i = 0; i < n; ++i) {
    ccld_hang_verdict v;
    std::memcpy(&v, host_blk.data() + o_out + i * sizeof(ccld_hang_verdict), sizeof v);
    v.roots = roots ? roots + (size_t)i * roots_stride : nullptr; v.roots_cap = roots ? roots_stride : 0;
    const u32 n_copy = std::min<u32>(std::min<u32>(v.n_roots_total, members[i]), v.roots_cap);
    if (n_copy) std::memcpy(v.roots, host_blk.data() + o_roots[i], n_copy * 4ull);
    out[i] = v;
    if (alerts) alerts[i] = al[i];
  }
  return CCLD_OK;
}

int ccld_get_optable(ccld_ctx* ctx, uint32_t window_id, ccld_optable* out) {
  if (!ctx || !out) return CCLD_ERR_ARG;
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  const WinDesc& d = w->d; const u64 G = d.n_groups;
  out->n_groups = G; out->n_slots = d.n_slots;
  const i64* gi = d.gi64; const u32* gu = d.gu32;
  out->e_min = gi + GI_E_MIN * G; out->arrival_skew = gi + GI_ARRIVAL_SKEW * G; out->t_max = gi + GI_T_MAX * G; out->t_min = gi + GI_T_MIN * G;
  out->span = gi + GI_SPAN * G; out->med_skew = gi + GI_MED_SKEW * G; out->mad_skew = gi + GI_MAD_SKEW * G;
  out->med_dur = gi + GI_MED_DUR * G; out->mad_dur = gi + GI_MAD_DUR * G;
  out->rank_tmin = gu + GU_RANK_TMIN * G; out->rank_tmax = gu + GU_RANK_TMAX * G; out->max_chg = gu + GU_MAX_CHG * G;
  out->rank_max_chg = gu + GU_RANK_MAX_CHG * G; out->n_present = gu + GU_N_PRESENT * G; out->gflags = gu + GU_GFLAGS * G;
  out->busbw = d.gbw; out->flags = d.flags; out->perm = d.perm;
  return CCLD_OK;
}

int ccld_get_ranges(ccld_ctx* ctx, uint32_t window_id, ccld_comm_range* rows, uint32_t cap, uint32_t* n_total) {
  if (!ctx || !n_total) return CCLD_ERR_ARG;
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  CK(cudaSetDevice(ctx->device));
  const u32 nc = ctx->reg.n_comms;
  std::vector<RangeRow> rr(nc);
  CK(cudaMemcpyAsync(rr.data(), w->d.ranges, nc * sizeof(RangeRow), cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  u32 k = 0;
  for (u32 c = 0; c < nc; ++c) {
    if (rr[c].n_seq == 0) continue;
    if (rows && k < cap) { rows[k].comm = ctx->comms[c].id; rows[k].n = rr[c].n; rows[k].seq_lo = rr[c].seq_lo; rows[k].n_seq = rr[c].n_seq;
                           rows[k].group0 = rr[c].group0; rows[k].slot0 = rr[c].slot0; }
    ++k;
  }
  *n_total = k;
  return CCLD_OK;
}

int ccld_get_rank_stats(ccld_ctx* ctx, uint32_t n_ranks, uint32_t* votes, uint32_t* ops, uint32_t* bw_cnt, double* bw_sum) {
  if (!ctx || !votes || !ops || !bw_cnt || !bw_sum) return CCLD_ERR_ARG;
  if (!ctx->finalized) return fail(ctx, CCLD_ERR_STATE, "nothing analysed yet");
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  CK(cudaSetDevice(ctx->device));
  std::memset(votes, 0, (size_t)n_ranks * 16); std::memset(ops, 0, (size_t)n_ranks * 4);
  std::memset(bw_cnt, 0, (size_t)n_ranks * 4); std::memset(bw_sum, 0, (size_t)n_ranks * 8);
  const u32 n = std::min(n_ranks, ctx->reg.n_ranks);
  cudaStream_t st = ctx->stream;
  CK(cudaMemcpyAsync(votes, ctx->reg.votes, (size_t)n * 16, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(ops, ctx->reg.ops, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(bw_cnt, ctx->reg.bw_cnt, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(bw_sum, ctx->reg.bw_sum, (size_t)n * 8, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return CCLD_OK;
}

int ccld_trace_attach_opset(ccld_ctx* ctx, uint32_t window_id, int mem_kind, const uint8_t* algo, const uint8_t* proto) {
  if (!ctx) return CCLD_ERR_ARG;
  if (mem_kind != 0 && mem_kind != 1) return fail(ctx, CCLD_ERR_ARG, "mem_kind must be 0 (host) or 1 (device)");
  auto it = ctx->windows.find(window_id);
  if (it == ctx->windows.end()) return fail(ctx, CCLD_ERR_NO_WINDOW, "unknown window id");
  WindowHost& w = it->second;
  if (w.n_rec > 0 && (!algo || !proto)) return fail(ctx, CCLD_ERR_ARG, "null column");
  CK(cudaSetDevice(ctx->device));
  if (w.owns_opset) { CK(cudaStreamSynchronize(ctx->stream)); ctx->pool.put(w.opset_own); w.owns_opset = false; }
  if (mem_kind == 1 || w.n_rec == 0) { w.algo = algo; w.proto = proto; return CCLD_OK; }
  cudaError_t e;
  const size_t half = align_up(w.n_rec);
  w.opset_own = ctx->pool.get(2 * half, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "window allocation failed");
  w.owns_opset = true;
  char* b = (char*)w.opset_own.p;
  CK(cudaMemcpyAsync(b, algo, w.n_rec, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaMemcpyAsync(b + half, proto, w.n_rec, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));       // the caller's host arrays are free again
  w.algo = (const u8*)b; w.proto = (const u8*)(b + half);
  return CCLD_OK;
}

int ccld_opset_check(ccld_ctx* ctx, uint32_t window_id, uint32_t comm, uint32_t seq, ccld_opset_verdict* out) {
  if (!ctx || !out) return CCLD_ERR_ARG;
  WindowHost* w;
  { int rc = find_analysed(ctx, window_id, &w); if (rc != CCLD_OK) return rc; }
  auto ci = ctx->comm_idx.find(comm);
  if (ci == ctx->comm_idx.end()) return fail(ctx, CCLD_ERR_UNKNOWN_COMM, "unknown communicator");
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->stream;
  const u32 n = (u32)ctx->comms[ci->second].ranks.size();
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up(off + b); return o; };
  const size_t o_hi = take(n * 8ull), o_lo = take(n * 4ull), o_rk = take(n * 4ull), o_out = take(sizeof(ccld_opset_verdict));
  cudaError_t e;
  Block blk = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "scratch allocation failed");
  char* b = (char*)blk.p;
  OpsetArgs A; A.c = ci->second; A.seq = seq; A.algo = w->algo; A.proto = w->proto;
  A.key_hi = (u64*)(b + o_hi); A.key_lo = (u32*)(b + o_lo); A.ranks = (u32*)(b + o_rk); A.ranks_cap = n; A.out = (ccld_opset_verdict*)(b + o_out);
  k_opset_check<<<1, 1024, 0, st>>>(w->d_desc, ctx->reg, A);
  ccld_opset_verdict v;
  u32* ranks = out->ranks; const u32 cap = ranks ? out->ranks_cap : 0;
  int rc = CCLD_OK;
  if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(&v, A.out, sizeof v, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) rc = CCLD_ERR_CUDA;
  if (rc == CCLD_OK) {
    *out = v; out->ranks = ranks; out->ranks_cap = cap;
    const u32 n_copy = std::min<u32>(std::min<u32>(v.n_deviating_total, n), cap);
    if (n_copy && (cudaMemcpyAsync(ranks, A.ranks, n_copy * 4ull, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)) rc = CCLD_ERR_CUDA;
  }
  ctx->pool.put(blk);
  if (rc != CCLD_OK) return fail(ctx, rc, "op-set check failed");
  return CCLD_OK;
}

namespace {
struct StateHeader { u64 magic; u32 version, n_comms, n_ranks, pad; u64 stats_bytes; };
constexpr u64 STATE_MAGIC = 0x3130545344434343ull;    // "CCCDST01"
}  // namespace

int ccld_state_export(ccld_ctx* ctx, void* buf, uint64_t cap, uint64_t* n_bytes) {
  if (!ctx || !n_bytes) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  { int rc = finalize_registry(ctx); if (rc != CCLD_OK) return rc; }
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  const u32 nc = ctx->reg.n_comms;
  const u64 need = sizeof(StateHeader) + (u64)nc * 12 + ctx->stats_bytes;
  *n_bytes = need;
  if (!buf || cap < need) return buf ? fail(ctx, CCLD_ERR_CAPACITY, "state buffer too small") : CCLD_OK;
  char* p = (char*)buf;
  StateHeader h{STATE_MAGIC, 1u, nc, ctx->n_ranks, 0u, (u64)ctx->stats_bytes};
  std::memcpy(p, &h, sizeof h); p += sizeof h;
  for (u32 c = 0; c < nc; ++c) { const u32 row[3] = {ctx->comms[c].id, (u32)ctx->comms[c].ranks.size(), ctx->comms[c].seq0}; std::memcpy(p, row, 12); p += 12; }
  CK(cudaMemcpyAsync(p, (char*)ctx->reg_blk.p + ctx->stats_off, ctx->stats_bytes, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  return CCLD_OK;
}

int ccld_state_import(ccld_ctx* ctx, const void* buf, uint64_t n_bytes) {
  if (!ctx || !buf) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  { int rc = finalize_registry(ctx); if (rc != CCLD_OK) return rc; }
  { int rc = settle(ctx); if (rc != CCLD_OK) return rc; }
  const u32 nc = ctx->reg.n_comms;
  StateHeader h;
  if (n_bytes < sizeof h) return fail(ctx, CCLD_ERR_ARG, "state blob too short");
  std::memcpy(&h, buf, sizeof h);
  if (h.magic != STATE_MAGIC || h.version != 1) return fail(ctx, CCLD_ERR_ARG, "not a state blob of this library version");
  if (h.n_comms != nc || h.n_ranks != ctx->n_ranks || h.stats_bytes != ctx->stats_bytes || n_bytes != sizeof h + (u64)nc * 12 + h.stats_bytes)
    return fail(ctx, CCLD_ERR_ARG, "state blob belongs to another set of communicators");
  const char* p = (const char*)buf + sizeof h;
  for (u32 c = 0; c < nc; ++c) {
    u32 row[3]; std::memcpy(row, p, 12); p += 12;
    if (row[0] != ctx->comms[c].id || row[1] != (u32)ctx->comms[c].ranks.size() || row[2] != ctx->comms[c].seq0)
      return fail(ctx, CCLD_ERR_ARG, "state blob belongs to another set of communicators");
  }
  CK(cudaStreamSynchronize(ctx->stream));
  CK(cudaMemcpyAsync((char*)ctx->reg_blk.p + ctx->stats_off, p, ctx->stats_bytes, cudaMemcpyHostToDevice, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  return CCLD_OK;
}

int ccld_derive_rates(ccld_ctx* ctx, uint64_t n_rec, const uint32_t* rank, const int64_t* t_enter_ns, const int64_t* t_exit_ns,
                      uint32_t n_ranks, uint64_t n_ticks, const uint64_t* tick_off, const int64_t* tick_ns,
                      const uint32_t* send_count, const uint32_t* recv_count, uint32_t* send_chg, uint32_t* recv_chg) {
  if (!ctx) return CCLD_ERR_ARG;
  if (n_rec && (!rank || !t_enter_ns || !t_exit_ns || !send_chg || !recv_chg)) return fail(ctx, CCLD_ERR_ARG, "null record column");
  if (n_ranks == 0 || !tick_off) return fail(ctx, CCLD_ERR_ARG, "tick_off is required (n_ranks + 1 entries)");
  if (n_ticks && (!tick_ns || !send_count || !recv_count)) return fail(ctx, CCLD_ERR_ARG, "null tick column");
  if (n_ticks >= 0xFFFFFFFFull) return fail(ctx, CCLD_ERR_CAPACITY, "too many ticks for 32-bit change counts");
  if ((n_rec + RT_THREADS - 1) / RT_THREADS > 0x7FFFFFFFull) return fail(ctx, CCLD_ERR_CAPACITY, "too many records for one launch");
  CK(cudaSetDevice(ctx->device));
  if (n_rec == 0) return CCLD_OK;
  cudaStream_t st = ctx->stream;
  const u64 n_tiles = (n_ticks + RT_TILE - 1) / RT_TILE;
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up(off + b); return o; };
  const size_t o_blk = take(((n_ticks + 31) / 32 + 1) * sizeof(TickBlock)), o_sum = take((n_tiles + 1) * 8);
  cudaError_t e;
  Block blk = ctx->pool.get(off, &e);
  if (e != cudaSuccess) return fail(ctx, CCLD_ERR_NOMEM, "scratch allocation failed");
  TickArgs A; A.n_ticks = n_ticks; A.n_ranks = n_ranks; A.tick_off = tick_off; A.tick_ns = tick_ns; A.send = send_count; A.recv = recv_count;
  A.blk = (TickBlock*)((char*)blk.p + o_blk); A.tile_sum = (u64*)((char*)blk.p + o_sum);
  if (n_tiles) {
    k_tick_blocks<<<(u32)n_tiles, RT_THREADS, 0, st>>>(A);
    k_tile_scan<<<1, TS_THREADS, 0, st>>>(A.tile_sum, n_tiles);
    k_block_prefix<<<(u32)n_tiles, RB_PER_TILE, 0, st>>>(A);
  }
  k_record_rates<<<(u32)((n_rec + RT_THREADS - 1) / RT_THREADS), RT_THREADS, 0, st>>>(A, n_rec, rank, t_enter_ns, t_exit_ns, send_chg, recv_chg);
  const cudaError_t le = cudaGetLastError();
  ctx->pool.put(blk);           // later work on this stream runs after these kernels: the block can be handed out again
  if (le != cudaSuccess) return fail(ctx, CCLD_ERR_CUDA, std::string("rate kernels: ") + cudaGetErrorString(le));
  return CCLD_OK;
}

int ccld_timing_enable(ccld_ctx* ctx, int on) {
  if (!ctx) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  CK(cudaStreamSynchronize(ctx->stream));
  if (on && ctx->ring.empty()) {
    ctx->ring.resize(TIMER_RING);
    for (auto& sl : ctx->ring) for (int i = 0; i < TIMER_PAIRS; ++i) { CK(cudaEventCreate(&sl.a[i])); CK(cudaEventCreate(&sl.b[i])); }
  }
  for (auto& sl : ctx->ring) sl.n = 0;
  std::memset(ctx->t_ms, 0, sizeof ctx->t_ms); std::memset(ctx->t_launches, 0, sizeof ctx->t_launches);
  ctx->timing = on != 0;
  return CCLD_OK;
}

int ccld_get_kernel_times(ccld_ctx* ctx, double* ms, uint64_t* launches) {
  if (!ctx || !ms || !launches) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  CK(cudaStreamSynchronize(ctx->stream));
  for (auto& sl : ctx->ring) timer_harvest(ctx, sl);
  for (int k = 0; k < CCLD_K_KINDS; ++k) { ms[k] = ctx->t_ms[k]; launches[k] = ctx->t_launches[k]; }
  return CCLD_OK;
}

int ccld_copy_to_host(ccld_ctx* ctx, void* dst_host, const void* src_device, uint64_t bytes) {
  if (!ctx || (bytes && (!dst_host || !src_device))) return CCLD_ERR_ARG;
  CK(cudaSetDevice(ctx->device));
  if (bytes) CK(cudaMemcpyAsync(dst_host, src_device, bytes, cudaMemcpyDeviceToHost, ctx->stream));
  CK(cudaStreamSynchronize(ctx->stream));
  return CCLD_OK;
}

}  // extern "C"
