/*
 * ccld.h - C ABI of the CCL-D decision-analyzer hot path on one NVIDIA B200 (sm_100a).
 *
 * The library analyses batches ("windows") of rank-level collective-communication trace records
 * the way the paper's centralized Decision Analysis Module does (Sec. 3, Sec. 4.2): it groups the
 * records by (communicator, operation counter) - the Trace ID of Sec. 5.1 -, reduces each group
 * across its ranks, tests every rank against the group with a robust median/MAD rule, keeps
 * per-rank anomaly votes, applies the slow-detection and slow-location rules of Eq. 1-4 per
 * communicator and window, raises hang alerts (Sec. 4.2.1) and locates the root rank of a hang
 * with the decision tree of Sec. 4.2.2 / Fig. 6 from per-channel SendCount/RecvCount counters.
 *
 * Conventions
 *   - Every function returns CCLD_OK (0) or a negative CCLD_ERR_* code; nothing throws or aborts.
 *     ccld_last_error() returns a text for the last failure on that context.
 *   - All compute runs in CUDA kernels on the context's device and stream. There is no CPU
 *     fallback: without a usable CUDA device ccld_create fails with CCLD_ERR_CUDA.
 *   - "host" / "device" is stated for every pointer. Output structs are caller-allocated PODs;
 *     variable-length lists have a caller-supplied capacity and a *_total count so truncation
 *     is visible.
 *   - Times are int64 nanoseconds; thresholds are integers in milli-units (x1000).
 *   - A context is not thread-safe; use one per thread or lock around it.
 */
#ifndef CCLD_H
#define CCLD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ccld_ctx ccld_ctx; /* opaque, library-owned */

enum {
  CCLD_OK = 0,
  CCLD_ERR_ARG = -1,          /* bad argument (null pointer, zero size, unsupported option) */
  CCLD_ERR_NOMEM = -2,        /* host or device allocation failed */
  CCLD_ERR_CUDA = -3,         /* a CUDA call failed; see ccld_last_error */
  CCLD_ERR_UNKNOWN_COMM = -4, /* a record names a communicator that was never registered */
  CCLD_ERR_NOT_MEMBER = -5,   /* a record's rank is not a member of its communicator */
  CCLD_ERR_SEQ_RANGE = -6,    /* a record's op counter is below the communicator's first one */
  CCLD_ERR_NO_WINDOW = -7,    /* unknown window id, or window not analysed yet */
  CCLD_ERR_CAPACITY = -8,     /* a size limit of the library was exceeded */
  CCLD_ERR_STATE = -9,        /* call order violated (e.g. window analysed twice) */
  CCLD_ERR_DUPLICATE = -10    /* two records with the same (communicator, op counter, rank) */
};

/* Operation types (the collectives of Sec. 2.1 plus point-to-point and broadcast). */
enum { CCLD_OP_ALLREDUCE = 0, CCLD_OP_ALLGATHER = 1, CCLD_OP_REDUCESCATTER = 2, CCLD_OP_ALLTOALL = 3,
       CCLD_OP_SENDRECV = 4, CCLD_OP_BROADCAST = 5 };

/* Per-slot flag byte (one per member of every group, in group-major order). */
enum { CCLD_F_SKEW_OUT = 1, CCLD_F_DUR_OUT = 2, CCLD_F_SKEW_HI = 4, CCLD_F_DUR_HI = 8,
       CCLD_F_MISSING = 64, CCLD_F_NOT_ANALYSED = 128 };

/* Per-group flag word. */
enum { CCLD_G_COMPLETE = 1, CCLD_G_INCOMPLETE = 2, CCLD_G_BARRIER = 4, CCLD_G_OPSET_MISMATCH = 8,
       CCLD_G_ANALYSED = 16, CCLD_G_HANG_ALERT = 32, CCLD_G_INFLIGHT = 64, CCLD_G_BAD_TIME = 128 };

/* Input error bits reported in ccld_verdict.error_bits. */
enum { CCLD_E_UNKNOWN_COMM = 1, CCLD_E_NOT_MEMBER = 2, CCLD_E_SEQ_RANGE = 4, CCLD_E_DUPLICATE = 8,
       CCLD_E_CAPACITY = 16 };

/* Limits. */
#define CCLD_MAX_COMM_SIZE 8192u          /* ranks per communicator */
#define CCLD_MAX_RANK_ID (1u << 22)       /* rank ids must be below this */
#define CCLD_MAX_ALERTS_PER_WINDOW 1024u  /* hang alerts kept per window (the total is counted) */

/*
 * Analysis parameters. Defaults (ccld_params_default) are the values the paper quotes:
 * theta_slow close to 3 (Sec. 4.2.1), alpha = 0.4 and beta = 0.6 (Sec. 4.2.2), m = min(100 rounds,
 * rounds of the first two minutes) (Sec. 4.2.1, Eq. 1), 5-minute hang threshold (Sec. 6.1),
 * barrier = AllReduce of fewer than 4 bytes (Sec. 4.2.1). tbase_init_ns is the administrator's
 * T_base^(init) of Eq. 1 and must be > 0. The remaining fields belong to the rank-level
 * median/MAD test, for which the paper gives no values.
 */
typedef struct {
  int64_t tbase_init_ns;       /* T_base^(init), Eq. 1 */
  uint32_t theta_slow_milli;   /* slow iff (T_max - T_base) * 1000 > theta_slow_milli * T_base, Eq. 3 */
  uint32_t alpha_milli;        /* P < alpha: communication-slow, Eq. 4 */
  uint32_t beta_milli;         /* P > beta: computation-slow, Eq. 4 */
  uint32_t m_max_rounds;       /* Eq. 1: at most this many rounds feed the baseline */
  int64_t m_max_ns;            /* Eq. 1: ... and only rounds that start within this time of the first */
  int64_t hang_ns;             /* hang alert iff now - t_enter > hang_ns for an in-flight record */
  uint64_t barrier_bytes;      /* AllReduce with bytes < barrier_bytes is a barrier */
  uint32_t slow_rep_threshold; /* location is triggered once the cumulative slow count exceeds this */
  uint32_t k_milli;            /* outlier iff |x - med| * 1000 > k_milli * MAD */
  uint32_t min_group;          /* groups with fewer ranks get no median/MAD test */
  uint32_t vote_rep_milli;     /* rank is a suspect iff votes * 1000 >= vote_rep_milli * ops */
} ccld_params;

void ccld_params_default(ccld_params* p /* host, out */);

/*
 * Lifecycle. `device` is a CUDA ordinal, `cuda_stream` a cudaStream_t (NULL = default stream) on
 * which every copy and kernel of this context is enqueued. The context owns all device memory it
 * allocates and frees it in ccld_destroy.
 */
int ccld_create(ccld_ctx** out, const ccld_params* params /* host */, int device, void* cuda_stream);
int ccld_destroy(ccld_ctx* ctx);
const char* ccld_last_error(ccld_ctx* ctx);

/*
 * Communicator registration (the "domain initialization" of Sec. 2.1): `ranks` (host, n entries,
 * copied) lists the members in ring order - position p sends to position p+1 mod n -, which the
 * hang localizer uses. `algo` 0 = ring, 1 = tree (other values: CCLD_ERR_ARG); a tree communicator
 * also needs ccld_comm_set_layers before its hangs can be located. `seq0` is the communicator's
 * first operation counter. All communicators must be registered before the first
 * ccld_analyze_window (later calls return CCLD_ERR_STATE). 1 <= n <= CCLD_MAX_COMM_SIZE.
 */
int ccld_comm_register(ccld_ctx* ctx, uint32_t comm, const uint32_t* ranks, uint32_t n, uint8_t algo, uint32_t seq0);

/*
 * Tree communicators (Sec. 4.2.1): the SendCount / RecvCount of two members are comparable only
 * when both sit in the same layer of the tree, so the diagnosis that compares them - branch H3 of
 * the hang decision tree - is restricted to same-layer members. `layer` (host, one entry per
 * member in the order given to ccld_comm_register, copied) names each member's layer; the ids are
 * arbitrary, equal id = same layer. For such a communicator ccld_locate_hang / ccld_locate_hangs
 * answer H3 like this: in every layer take the gap between the largest and the smallest counter
 * total; the root is the member holding the minimum of the layer with the widest gap (equal gaps,
 * or several holders: the lowest position); if no layer disagrees with itself n_roots_total = 0
 * and min_total = 0. The same restriction holds for the update frequencies: the root_comm of a
 * slowed tree communicator (ccld_comm_verdict) is the member whose change count in the selected
 * round - the larger of its two rate columns - lies furthest above the smallest of its layer
 * (equal excesses: the lowest position); if no layer disagrees with itself, or the window has no
 * rate columns, the member with the longest duration stands in (rate_source = 1). H1, H2 and the
 * per-operation statistics (which compare times, not counters) treat a tree communicator like a
 * ring; so does root_comm while the layers are not set. Errors: CCLD_ERR_STATE after the first analysis,
 * CCLD_ERR_UNKNOWN_COMM, CCLD_ERR_ARG for a ring communicator or a null pointer. Locating a hang
 * on a tree communicator whose layers were never set returns CCLD_ERR_STATE.
 */
int ccld_comm_set_layers(ccld_ctx* ctx, uint32_t comm, const uint32_t* layer);

/*
 * Hands one window of trace records to the analyzer - what the rank probes push on kernel
 * completion (Sec. 5.2, step 4). SoA columns of length n_rec, any record order:
 *   rank, comm, seq   uint32   reporting rank, communicator id, operation counter (Trace ID, Sec. 5.1)
 *   op                uint8    CCLD_OP_*
 *   bytes             uint64   message size (Operation Type Set, Sec. 4.1.2)
 *   t_enter, t_exit   int64    ns; t_exit = -1 marks an operation still in flight
 *   send_chg,recv_chg uint32   observed SendCount/RecvCount value changes during the op, i.e.
 *                              1/SendRate and 1/RecvRate of Sec. 4.1.2; both may be NULL
 * Optional progress frames (n_frames may be 0): for frame f, rank f_rank[f] reports for op
 * (f_comm[f], f_seq[f]) the counters progress[f][channel][0] = SendCount and [1] = RecvCount
 * (Probing Frame body, Sec. 5.1), n_channels channels per frame.
 * mem_kind 0: every pointer is host memory; the data is copied to the device with asynchronous
 * copies on the context's stream. Pageable buffers may be reused when the call returns; pinned
 * buffers must stay unchanged until the stream has passed the copies (any synchronizing call of
 * this library, e.g. ccld_get_verdict, guarantees that).
 * mem_kind 1: every pointer is device memory on the context's device, borrowed until
 * ccld_window_release or ccld_destroy; the caller keeps it alive and unchanged.
 * At most one (comm, seq, rank) record per window (else CCLD_E_DUPLICATE at the verdict).
 * n_rec < 2^32 - 1. A window id may be uploaded once until released.
 */
int ccld_trace_upload(ccld_ctx* ctx, uint32_t window_id, uint64_t n_rec, int mem_kind,
                      const uint32_t* rank, const uint32_t* comm, const uint32_t* seq, const uint8_t* op,
                      const uint64_t* bytes, const int64_t* t_enter_ns, const int64_t* t_exit_ns,
                      const uint32_t* send_chg, const uint32_t* recv_chg,
                      uint32_t n_frames, const uint32_t* f_rank, const uint32_t* f_comm, const uint32_t* f_seq,
                      uint32_t n_channels, const uint32_t* progress);

/* Drops a window: its records (if copied) and its results. */
int ccld_window_release(ccld_ctx* ctx, uint32_t window_id);

/*
 * Analyses windows first_window .. first_window + n_windows - 1 (all uploaded, none analysed yet),
 * in that order: grouping by (communicator, op counter) (Sec. 4.2.1), per-op cross-rank
 * reductions, median/MAD flags, votes, then per communicator the window rules of Eq. 1-4 whose
 * state (baseline rounds, slow counter) carries from window to window. `now_ns` is the analyzer's
 * clock for the hang test. Work is enqueued on the context's stream.
 * The first batch of a shape (the same record count in every window) waits, in the middle of the
 * call, for one short device round trip that sizes the result buffers. A later batch of the same
 * shape does not wait at all: its buffers are sized from the totals the shape had before, the
 * call only enqueues and returns, and the layout pass checks the totals on the device. If they
 * differ, that batch and every batch enqueued after it give up on the device without touching any
 * state, and the next call that synchronizes anyway (ccld_get_verdict and the other result
 * accessors, ccld_window_release, ccld_state_export, a batch of a new shape) analyses them again
 * in order, this time waiting - results and their order are the same either way, only the time
 * differs. ccld_set_speculation(ctx, 0) makes every call wait.
 * A window is refused (CCLD_E_CAPACITY in its verdict, nothing analysed) if the op counters seen
 * in it would need more than 2 * n_rec + (sum of communicator sizes) slots. A batch holds at most
 * 65,535 windows (CCLD_ERR_CAPACITY beyond).
 */
int ccld_analyze_window(ccld_ctx* ctx, uint32_t first_window, uint32_t n_windows, int64_t now_ns);

/*
 * Whether ccld_analyze_window may size a batch from the totals its shape had before instead of
 * waiting for the layout pass (Sec. 4.2.1 analyses one window per minute: a monitoring loop sees
 * the same shape over and over). on = 0: always wait; on = 1 (the default): wait only for shapes
 * not seen before. Batches still in doubt are settled first.
 */
int ccld_set_speculation(ccld_ctx* ctx, int on);

/* Clears votes, per-communicator state and all window results (records stay uploaded). */
int ccld_reset(ccld_ctx* ctx);

/* One suspect rank: kind 1 = straggler (late arrivals), 2 = slow link (long durations). */
typedef struct {
  uint32_t kind, rank, votes, ops;
  double mean_busbw; /* bytes/ns = GB/s, mean over the rank's complete non-barrier ops */
} ccld_suspect;

/* Slow detection / location of one communicator in one window (Sec. 4.2.1-4.2.2). */
typedef struct {
  uint32_t comm;            /* communicator id */
  uint32_t n_rounds;        /* complete non-barrier rounds of this window */
  uint32_t sel_seq;         /* round selected by Eq. 2 (0xFFFFFFFF if none) */
  uint32_t cls;             /* 0 none, 1 computation-slow, 2 communication-slow, 3 mixed */
  uint32_t slow_detected;   /* R > theta_slow, Eq. 3 */
  uint32_t located;         /* slow_detected and the repetition counter exceeded its threshold */
  uint32_t baseline_static; /* 1: T_base is still the configured value (slow-at-start) */
  uint32_t rate_source;     /* 0: root_comm from the rate columns, 1: longest duration stands in */
  uint32_t root_comp;       /* rank with minimal duration in the selected round (0xFFFFFFFF if not slow) */
  uint32_t root_comm;       /* rank with minimal Send/Recv rate in the selected round */
  uint64_t slow_count;      /* cumulative slow detections of this communicator */
  uint64_t rounds_total;    /* rounds seen so far (r of Eq. 1) */
  uint64_t m;               /* m of Eq. 1, 0 while not fixed */
  int64_t t_max, t_min, t_base;
  double R, P;              /* Eq. 3, Eq. 4 (P = 0 when not slow) */
} ccld_comm_verdict;

typedef struct {
  uint32_t comm, seq;
  int64_t age_ns; /* now - t_enter of the oldest in-flight member */
} ccld_hang_alert;

/*
 * Result of one analysed window plus the cumulative suspect list. The caller sets the three
 * pointers (host memory, may be NULL with capacity 0) and capacities; the library fills the
 * rest. comm_rows are ordered by registration order of the communicators, alerts by
 * (communicator registration order, seq), suspects by (kind, votes descending, rank).
 */
typedef struct {
  uint64_t n_records, n_groups, n_slots, n_rejected, n_complete, n_incomplete, n_barrier, n_analysed,
      n_flag_skew, n_flag_dur, n_opset_mismatch;
  uint32_t error_bits; /* CCLD_E_* seen in this window */
  uint32_t n_comm_rows_total, n_alerts_total, n_suspects_total;
  ccld_comm_verdict* comm_rows; uint32_t comm_rows_cap;
  ccld_hang_alert* alerts;      uint32_t alerts_cap;
  ccld_suspect* suspects;       uint32_t suspects_cap;
} ccld_verdict;

/*
 * Synchronizes the stream and returns the verdict of an analysed window. Returns CCLD_OK, or the
 * CCLD_ERR_* that corresponds to the lowest set bit of error_bits (the struct is filled either way).
 */
int ccld_get_verdict(ccld_ctx* ctx, uint32_t window_id, ccld_verdict* out /* host */);

/*
 * Hang location (Sec. 4.2.2, Fig. 6) for op (comm, seq) as seen in window `window_id`:
 *   H1 (cls 1): members with no record of an op counter >= seq - they never entered; roots = those.
 *   H2 (cls 2): all entered, some members' record of `seq` is complete - roots = those non-hung ranks.
 *   H3 (cls 3): all hung - root = the member with the fewest SendCount+RecvCount summed over channels;
 *       among equal minima the one whose ring predecessor has made more progress, then the lowest
 *       ring position. A member without a frame counts as zero progress.
 * roots (host, caller-allocated, may be NULL) receives up to roots_cap rank ids in ring order.
 * Synchronizes the stream.
 */
typedef struct {
  uint32_t cls, n_roots_total, n_not_entered, n_hung, n_not_hung, n_missing_frames;
  uint32_t stuck_step; /* H3: the root's smallest RecvCount over channels */
  uint32_t n_members;
  uint64_t min_total;  /* H3: the root's summed counters */
  uint32_t* roots; uint32_t roots_cap;
} ccld_hang_verdict;

int ccld_locate_hang(ccld_ctx* ctx, uint32_t window_id, uint32_t comm, uint32_t seq, ccld_hang_verdict* out /* host */);

/*
 * Hang location for every alert of an analysed window in one kernel launch (Sec. 4.2.2, Fig. 6: the decision tree runs
 * for each hang that detection reported; Sec. 4.2.1 raises the alerts). out[i] is what ccld_locate_hang returns for the
 * i-th alert in the order ccld_get_verdict lists them (communicator registration order, then op counter).
 *   alerts  host, cap entries, may be NULL: receives the (comm, seq, age) that out[i] belongs to
 *   out     host, cap entries: the verdicts; out[i].roots is set to roots + i * roots_stride, out[i].roots_cap to
 *           roots_stride (NULL and 0 when roots is NULL)
 *   roots   host, cap * roots_stride rank ids, may be NULL
 *   n_total the window's number of alerts; at most min(cap, CCLD_MAX_ALERTS_PER_WINDOW) are located
 * Synchronizes the stream. Scratch comes from the context's block pool (CCLD_ERR_NOMEM if that fails).
 */
int ccld_locate_hangs(ccld_ctx* ctx, uint32_t window_id, ccld_hang_alert* alerts /* host */, ccld_hang_verdict* out /* host */,
                      uint32_t cap, uint32_t* roots /* host */, uint32_t roots_stride, uint32_t* n_total);

/*
 * Parity / inspection access to the per-op table of an analysed window. Device pointers, valid
 * until the window is released or the context reset. Groups are ordered by (communicator
 * registration order, seq); group g of communicator row r covers slots
 * [slot0_r + (g - group0_r) * n_r, ... + n_r). Column semantics (complete groups; zeros otherwise):
 *   e_min = min t_enter; arrival_skew = max (t_enter - e_min); t_max, t_min = max, min duration;
 *   span = max t_exit - e_min; med_x and mad_x = lower median and lower-median absolute deviation of
 *   skew and duration (analysed groups); rank_tmin, rank_tmax = ranks of min, max duration (ties:
 *   lowest ring position); max_chg, rank_max_chg = most observed count changes and its rank;
 *   busbw = bytes * f / span in bytes per ns with f = 2(n-1)/n allreduce, (n-1)/n allgather,
 *   reducescatter, alltoall, 1 otherwise.
 * perm holds, per slot, the index of the record in the uploaded columns (0xFFFFFFFF if the member is
 * missing). Unlike flags it is member-major inside a communicator: the record of ring position p and op
 * counter s of communicator row r is perm[slot0_r + p * n_seq_r + (s - seq_lo_r)].
 */
typedef struct {
  uint64_t n_groups, n_slots;
  const int64_t *e_min, *arrival_skew, *t_max, *t_min, *span, *med_skew, *mad_skew, *med_dur, *mad_dur;
  const uint32_t *rank_tmin, *rank_tmax, *max_chg, *rank_max_chg, *n_present, *gflags;
  const double* busbw;
  const uint8_t* flags;  /* [n_slots] */
  const uint32_t* perm;  /* [n_slots] */
} ccld_optable;

int ccld_get_optable(ccld_ctx* ctx, uint32_t window_id, ccld_optable* out /* host struct, device pointers */);

/* Per communicator of a window: which op counters it covers and where its groups and slots start. */
typedef struct {
  uint32_t comm, n, seq_lo, n_seq;
  uint64_t group0, slot0;
} ccld_comm_range;

/* Copies up to cap rows (host, registration order, only communicators with records); returns the total in *n_total. Synchronizes. */
int ccld_get_ranges(ccld_ctx* ctx, uint32_t window_id, ccld_comm_range* rows /* host */, uint32_t cap, uint32_t* n_total);

/*
 * Cumulative per-rank statistics for ranks [0, n_ranks): votes[r][4] = {skew high, skew low,
 * duration high, duration low}, ops = analysed ops, bw_cnt and bw_sum = count and fp64 sum of the
 * rank's per-op bus bandwidth. Host arrays, caller-allocated. Synchronizes.
 */
int ccld_get_rank_stats(ccld_ctx* ctx, uint32_t n_ranks, uint32_t* votes, uint32_t* ops, uint32_t* bw_cnt, double* bw_sum);

/*
 * Operation Type Set consistency (Sec. 4.1.2: each rank records the communication algorithm, protocol, data size and
 * operation name of an op, which stay constant during the communication; Sec. 4.2.2: inconsistent operations are the
 * cause that the not-hung ranks of hang leaf H2 point at).
 *   ccld_trace_attach_opset adds the two columns that ccld_trace_upload does not take - algorithm and protocol codes per
 *     record, in the order of the uploaded columns, n_rec entries each; host memory is copied, device memory borrowed
 *     until the window is released. Without it both count as 0. The window must have been uploaded.
 *   ccld_opset_check, for op (comm, seq) of an analysed window: the most frequent (op, bytes, algo, proto) among the
 *     members that reported the op - ties go to the tuple whose first holder stands earliest in the ring - how many
 *     members carry it, and the ranks that carry another tuple, in ring order, up to ranks_cap of them into out->ranks
 *     (host, caller-allocated, may be NULL). Synchronizes the stream.
 */
typedef struct {
  uint32_t n_members, n_present, n_deviating_total, majority_count;
  uint8_t op, algo, proto, pad;  /* the majority tuple (zeros if no member reported the op) */
  uint64_t bytes;
  uint32_t* ranks; uint32_t ranks_cap;
} ccld_opset_verdict;

int ccld_trace_attach_opset(ccld_ctx* ctx, uint32_t window_id, int mem_kind, const uint8_t* algo, const uint8_t* proto);
int ccld_opset_check(ccld_ctx* ctx, uint32_t window_id, uint32_t comm, uint32_t seq, ccld_opset_verdict* out /* host */);

/*
 * Cumulative analyzer state as a host blob: per communicator the Eq. 1 baseline state (rounds seen, first enter time, sum of
 * the first m T_max, m) and the repetition counter of slow detections (Sec. 4.2.1), per rank the vote counters, analysed-op
 * counts and bus-bandwidth sums. An analyzer service that restarts, or hands a job to another GPU, exports the state and
 * imports it into a context with the same communicators registered in the same order (ids, sizes and first counters are
 * checked; member lists are the caller's responsibility), then goes on with the next window as if nothing had happened.
 *   ccld_state_export: *n_bytes receives the blob size; with buf = NULL only the size is returned. cap < size with a
 *     buffer gives CCLD_ERR_CAPACITY. Synchronizes the stream.
 *   ccld_state_import: replaces the context's cumulative state; CCLD_ERR_ARG if the blob is malformed or belongs to
 *     another set of communicators. Synchronizes the stream.
 * Both fix the set of communicators (like the first ccld_analyze_window). Windows and their results are not part of it.
 */
int ccld_state_export(ccld_ctx* ctx, void* buf /* host */, uint64_t cap, uint64_t* n_bytes);
int ccld_state_import(ccld_ctx* ctx, const void* buf /* host */, uint64_t n_bytes);

/*
 * SendRate / RecvRate inputs from raw probe samples (Sec. 4.1.2: the rate is the reciprocal of the number of changes of
 * SendCount / RecvCount seen by a probe that samples at a fixed period; Sec. 5.2 step 2 has the host's diagnostic
 * thread derive it). This call does that step on the GPU and produces the send_chg / recv_chg columns that
 * ccld_trace_upload takes.
 *   Samples: rank r < n_ranks owns ticks [tick_off[r], tick_off[r + 1]) of tick_ns / send_count / recv_count, in time
 *   order; tick_off has n_ranks + 1 entries, tick_off[0] = 0, tick_off[n_ranks] = n_ticks.
 *   Result: for record i of rank r, send_chg[i] = the number of r's ticks k, other than r's first, with
 *   t_enter_ns[i] < tick_ns[k] <= t_end whose send_count differs from the previous tick's; t_end = t_exit_ns[i], or
 *   unbounded while the op is in flight (t_exit_ns[i] = -1). recv_chg likewise. A rank without ticks, or a rank id
 *   >= n_ranks, gets 0.
 * Every pointer is device memory of the context's device, owned by the caller and left untouched except for the two
 * outputs (n_rec entries each). The kernels are enqueued on the context's stream and the call returns without
 * synchronizing; scratch (8 bytes per tick) comes from the context's block pool. Counts are 32-bit:
 * n_ticks >= 2^32 - 1 is refused with CCLD_ERR_CAPACITY. Other errors: CCLD_ERR_ARG (null pointers, n_ranks = 0),
 * CCLD_ERR_NOMEM, CCLD_ERR_CUDA.
 */
int ccld_derive_rates(ccld_ctx* ctx, uint64_t n_rec, const uint32_t* rank, const int64_t* t_enter_ns, const int64_t* t_exit_ns,
                      uint32_t n_ranks, uint64_t n_ticks, const uint64_t* tick_off, const int64_t* tick_ns,
                      const uint32_t* send_count, const uint32_t* recv_count, uint32_t* send_chg, uint32_t* recv_chg);

/*
 * Per-kernel device timing for benchmarks. While enabled, ccld_analyze_window brackets each of its
 * kernel launches with CUDA events on the context's stream. ccld_get_kernel_times synchronizes the
 * stream and returns, per kernel kind, the summed device time in milliseconds and the number of
 * launches since timing was last enabled. Kinds: 0 op-counter range, 1 slot layout and work lists
 * (two launches per call), 2 slot scatter, 3 reductions n <= 128 (fused), 4 reductions n <= 1024,
 * 5 reductions n > 1024, 6 window decision. Enabling (on = 1) clears the sums; on = 0 stops timing.
 * Independently of this switch, every entry point and every stage of ccld_analyze_window opens a named NVTX range
 * ("ccld_analyze_window", "ccld: slot scatter", ...) on the calling thread, which costs nothing unless a timeline
 * tool is attached.
 */
#define CCLD_K_KINDS 7
int ccld_timing_enable(ccld_ctx* ctx, int on);
int ccld_get_kernel_times(ccld_ctx* ctx, double* ms /* host [CCLD_K_KINDS] */, uint64_t* launches /* host [CCLD_K_KINDS] */);

/*
 * Hang location for one ring without any allocation. The paper has no counterpart to this entry
 * point; it exists for callers that cannot allocate device memory when they need a diagnosis: a
 * watchdog thread looking at a job whose memory is exhausted or whose allocator sits behind the
 * hang itself, a plugin hosted inside another process that must leave that process's memory pool
 * alone, or a monitoring loop in which an allocation could stall the device. It needs no context and
 * calls no cudaMalloc, cudaFree or allocating library routine; its working memory is one fixed array
 * of CCLD_STATIC_SCRATCH_BYTES bytes inside the library's device image, so every GPU on which the
 * library has been used holds that much until the process exits.
 *
 * Set-up call. The CUDA runtime creates a device's primary context and loads the library's device
 * image (the array and the kernel) lazily, the first time a call names that device; that one-time
 * step does take device memory and fails with CCLD_ERR_NOMEM or CCLD_ERR_CUDA when none is left.
 * The first call on a device also looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and caches it. So make one call per device at start-up, while memory is
 * still available and before any stream capture begins (a one-member ring is enough); only the
 * calls after it allocate nothing. This is an ordinary host function: call it from a thread, not
 * from a signal handler.
 *
 * Inputs (all device memory on `device`, owned by the caller), indexed by ring position p < n_members:
 *   ranks[p]       rank id of the member at position p (position p sends to p+1 mod n)
 *   state[p]       bit0: the member entered the op (reported this or a later op counter),
 *                  bit1: its record of the op is complete (not hung), bit2: it has a progress frame
 *   progress[p][channel][0..1]  SendCount, RecvCount per channel (read only where bit2 is set;
 *                  may be NULL when n_channels is 0)
 * Output: *out (host) as for ccld_locate_hang - same classes H1/H2/H3, same tie-breaks, roots in ring
 * order into out->roots (host, caller-allocated, up to out->roots_cap). The call enqueues one kernel on
 * `cuda_stream` and synchronizes that stream before it returns.
 *
 * Limits and rules: n_members <= CCLD_STATIC_MAX_MEMBERS, else CCLD_ERR_CAPACITY and nothing runs.
 * `err` (host, may be NULL) receives a message of at most err_cap bytes on failure. All calls on a
 * device share the array, which keeps the previous call's contents; the kernel rewrites every entry it
 * reads, but calls whose kernels overlap on the GPU (other streams or host threads) race and must be
 * serialized by the caller. The caller's current device is restored on return.
 */
#define CCLD_STATIC_MAX_MEMBERS 8192u
#define CCLD_STATIC_SCRATCH_BYTES (CCLD_STATIC_MAX_MEMBERS * 12u + 256u)
int ccld_ring_locate_static(int device, void* cuda_stream, uint32_t n_members, const uint32_t* ranks /* device */,
                            const uint8_t* state /* device */, uint32_t n_channels, const uint32_t* progress /* device */,
                            ccld_hang_verdict* out /* host */, char* err /* host */, uint32_t err_cap);

/* Utility for inspection tools: synchronous copy of `bytes` bytes from device memory of this context to host memory. */
int ccld_copy_to_host(ccld_ctx* ctx, void* dst_host, const void* src_device, uint64_t bytes);

#ifdef __cplusplus
}
#endif
#endif /* CCLD_H */
