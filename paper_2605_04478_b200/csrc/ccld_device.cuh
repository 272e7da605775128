// Device-side data layout shared by the kernels and the host API of libccld (sm_100a).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/ccld.h"

namespace ccld {

typedef int64_t i64;
typedef uint64_t u64;
typedef uint32_t u32;
typedef uint8_t u8;
typedef unsigned long long ull;

constexpr u32 NONE = 0xFFFFFFFFu;
constexpr u64 U64_MAX_ = ~0ull;

// ---- launch geometry ----
constexpr int REC_THREADS = 128;       // record-streaming kernels: threads per CTA
constexpr int REC_PER_THREAD = 16;     //   each walks a run of consecutive records
constexpr int REC_PER_CTA = REC_THREADS * REC_PER_THREAD;
constexpr int SMALL_N = 8;             // communicators of up to 8 ranks: one thread per group
constexpr int SMALL_SEQS = 256;        //   threads per CTA: eight warps, each on a warp-tile of up to 32 op counters at a time
#ifndef CCLD_FUSED_WT_PER_CTA
#define CCLD_FUSED_WT_PER_CTA 16
#endif
constexpr u32 FUSED_WT_PER_CTA = CCLD_FUSED_WT_PER_CTA;   //   warp-tiles a CTA works through (a multiple of its eight warps)
constexpr int WARP_N = 128;            // up to 128 ranks: one warp per group, bitonic sort in registers
constexpr int MID_N = 1024;            // up to 1024 ranks: shared-memory bitonic sort, several groups per CTA
constexpr int MID_THREADS = 256;
constexpr int MID_ELEMS = 2048;        //   padded records per tile
constexpr int LARGE_SEQS = 8;          // above: tiles of up to 8 consecutive op counters (as many as fit shared memory), radix select
constexpr int LG_THREADS = 512;
constexpr int LG_WARPS = LG_THREADS / 32;
constexpr int LG_KEYS = 16;            //   (member, group) pairs a thread of the kernel holds at most
constexpr int LS_THREADS = 256;        //   staging kernel: a CTA takes LS_MEMBERS members of a tile
constexpr int LS_MEMBERS = 512;

struct Params {
  i64 tbase_init_ns, m_max_ns, hang_ns;
  u64 barrier_bytes;
  u32 theta_slow_milli, alpha_milli, beta_milli, m_max_rounds, slow_rep_threshold, k_milli, min_group, vote_rep_milli;
};

// Eq. 1 state of one communicator, carried from window to window.
struct CommState { u64 rounds; i64 t_first; i64 sum_m; u64 m; u64 slow_count; };

// Registered communicators (immutable after the first analysis) and cumulative per-rank statistics.
struct Registry {
  u32 n_comms, hash_mask, n_ranks, pad;
  const uint4* hash;        // open addressing: (communicator id, index, seq0, n), index NONE = empty
  const uint4* rank_tab;    // [n_ranks][2]: up to RANK_TAB_K inline (communicator id, index << 13 | position) pairs of a rank
  const u32* comm_id;       // [n_comms]
  const u32* comm_n;        // [n_comms] members
  const u32* comm_seq0;     // [n_comms]
  const u64* comm_moff;     // [n_comms] offset of the member list in `members`
  const u32* members;       // rank ids, ring order
  const u32* rank_ptr;      // [n_ranks+1] CSR over (communicator index, position) pairs of a rank
  const u32* ent_comm;
  const u32* ent_pos;
  CommState* state;         // [n_comms]
  u32* votes;               // [n_ranks][4] skew hi, skew lo, dur hi, dur lo
  u32* ops;                 // [n_ranks]
  u32* bw_cnt;              // [n_ranks]
  double* bw_sum;           // [n_ranks]
};

// rank_tab: pairs beyond RANK_TAB_K do not fit inline; the last pair then holds (NONE, RANK_TAB_OVERFLOW) and the
// CSR lists are searched instead. Empty pairs are (NONE, NONE).
constexpr int RANK_TAB_K = 4;
constexpr u32 RANK_TAB_OVERFLOW = 0xFFFFFFFEu;
constexpr u32 RANK_TAB_POS_BITS = 13;  // positions < CCLD_MAX_COMM_SIZE = 8192

// Which op counters a communicator covers in a window and where its groups / slots start.
// tile0 / n_units: where the communicator's TileSum entries start (index into its summary array) and how many it has.
struct RangeRow { u32 seq_lo, n_seq, row_idx, n; u64 group0, slot0; u32 tile0, n_units; };

enum { C_REJECTED = 0, C_COMPLETE, C_INCOMPLETE, C_BARRIER, C_ANALYSED, C_FLAG_SKEW, C_FLAG_DUR, C_MISMATCH,
       C_PRESENT, C_ALERTS, C_ERR, C_INTERNAL, C_COUNT = 16 };
constexpr int N_CLASSES = 4;           // reduction code paths: n <= 8, <= 128, <= 1024, larger
// Classes 0 and 1 run in one fused kernel whose work list is ordered by (window, time chunk): a window's op
// counters are cut into T chunks per communicator, so that the tiles of one chunk - which gather from the same
// stretch of every rank's records - run together and share the fetched sectors in L2.
constexpr u32 CHUNK_REF = 96;          // op counters per chunk of the busiest communicator of a window
constexpr u32 CHUNK_MAX = 64;          // at most this many chunks per window (longer chunks beyond)
enum { T_GROUPS = 0, T_SLOTS, T_FCTA, T_FWT, T_FSUM, T_TILES2, T_TILES3, T_ROWS, T_FAILED, T_CHUNKS, T_COUNT = 12 };
constexpr u64 FAILED_CAPACITY = 1, FAILED_EXPECT = 2;      // T_FAILED: the window needs too many slots / its layout is not the expected one
enum { B_FCTA = 0, B_FWT, B_FSUM, B_T2, B_T3, B_COUNT };

struct Tile { u32 w, c, seq_off, count; };                 // classes 2 and 3: one CTA each; summary index = tile index
// Work-list entries of the fused kernel carry a copy of the communicator's range row and member-list offset, so that a
// tile needs no further lookups before its first gather.
struct WarpTile { u32 c, seq_off, count, sum_idx; RangeRow row; u64 moff; };      // class 0: up to 32 consecutive op counters of one communicator
struct FusedCta { u32 w, cls, c, seq_off, count, sum_idx, wt_first, wt_count; RangeRow row; u64 moff; };   // class 0: wt_*; class 1: c .. sum_idx, row, moff

// What a tile contributes to its communicator's window decision (Eq. 2 and the round counts).
struct TileSum { u64 best_rng; u32 best_k, n_rounds, n_an, pad; };   // best_k: op-counter offset in the range, NONE if no round

// One window of a batch: input columns, scratch and result pointers (all device memory).
struct WinDesc {
  const u32 *rank, *comm, *seq;
  const u8* op;
  const u64* bytes;
  const i64 *t_enter, *t_exit;
  const u32 *send_chg, *recv_chg;   // may be null
  u64 n_rec;
  u64 slot_cap;                      // plan fails the window if it would need more slots
  u32 cta0, n_cta;                   // this window's CTAs in the record-streaming grids
  u32 *rmin, *rmax;                  // [n_comms] op counter range seen
  RangeRow* ranges;                  // [n_comms]
  uint4* srow;                       // [n_comms] scatter rows: first slot low, high, op counters covered (0 = nothing to place), first op counter
  uint4* rent;                       // [n_ranks][RANK_TAB_K] a rank's inline pairs resolved for this window: (communicator id, op counters
                                     //   covered (0: unused), first op counter, first slot of the member's column); 32-bit slots only
  u64* totals;                       // [T_COUNT]
  const u64* expect;                 // [T_COUNT] totals the host sized this window's results for without waiting (null: it waited)
  u32* poison;                       // set once a window's layout differs from what the host expected: every window planned later gives up too
  u64* counters;                     // [C_COUNT]
  // sized after the plan:
  u64 n_groups, n_slots;
  u32* perm;                         // [n_slots]
  u8* flags;                         // [n_slots]
  u32 *skey, *dkey;                  // [n_slots] staged 32-bit keys of the largest communicators (null when the batch has none)
  i64* gi64;                         // [9][n_groups]
  u32* gu32;                         // [6][n_groups]
  double* gbw;                       // [n_groups]
  ccld_comm_verdict* comm_rows;      // [n_rows]
  ccld_hang_alert* alerts;           // [CCLD_MAX_ALERTS_PER_WINDOW]
  u32 base[B_COUNT];                 // this window's first entry in the batch-wide lists (B_*)
  u32 pad;
  TileSum* tsum[3];                  // tile summaries of the whole batch: fused classes, class 2, class 3
};

enum { GI_E_MIN = 0, GI_ARRIVAL_SKEW, GI_T_MAX, GI_T_MIN, GI_SPAN, GI_MED_SKEW, GI_MAD_SKEW, GI_MED_DUR, GI_MAD_DUR, GI_COUNT };
enum { GU_RANK_TMIN = 0, GU_RANK_TMAX, GU_MAX_CHG, GU_RANK_MAX_CHG, GU_N_PRESENT, GU_GFLAGS, GU_COUNT };

__host__ __device__ inline u32 next_pow2(u32 n) { u32 p = 1; while (p < n) p <<= 1; return p; }
__host__ __device__ inline u32 comm_class(u32 n) { return n <= SMALL_N ? 0u : (n <= WARP_N ? 1u : (n <= MID_N ? 2u : 3u)); }
__host__ __device__ inline u32 mid_npad(u32 n) { u32 p = next_pow2(n); return p < 32 ? 32 : p; }
// Communicators of more than MID_N ranks: a tile is LARGE_SEQS consecutive op counters; the select kernel works on G of
// them side by side, as many as let a thread keep its share of the keys (at most LG_KEYS) in registers.
__host__ __device__ inline u32 large_npad(u32 n) { return (n + 31u) & ~31u; }
__host__ __device__ inline u32 large_g(u32 n) {
  u32 G = LARGE_SEQS;
  while (G > 1 && (u64)G * large_npad(n) > (u64)LG_KEYS * LG_THREADS) G >>= 1;
  return G;
}
// op counters per work unit: a warp-tile (class 0) or a CTA tile (classes 1 to 3)
__host__ __device__ inline u32 tile_seqs(u32 n) {
  u32 c = comm_class(n);
  return c == 0 ? 32u : (c <= 2 ? MID_ELEMS / mid_npad(n) : (u32)LARGE_SEQS);
}
__host__ __device__ inline u32 ceil_div(u32 a, u32 b) { return (a + b - 1) / b; }
// chunking of a fused-class communicator with n_seq op counters in a window of T chunks
__host__ __device__ inline u32 chunk_len(u32 n_seq, u32 T) { return ceil_div(n_seq, T); }
__host__ __device__ inline u32 chunk_count(u32 n_seq, u32 T) { return n_seq ? ceil_div(n_seq, chunk_len(n_seq, T)) : 0u; }
__host__ __device__ inline u32 chunk_size(u32 n_seq, u32 T, u32 tau) {    // op counters in chunk tau (0 beyond the last)
  const u32 S = chunk_len(n_seq, T);
  return (u64)tau * S >= n_seq ? 0u : (n_seq - tau * S < S ? n_seq - tau * S : S);
}

}  // namespace ccld
