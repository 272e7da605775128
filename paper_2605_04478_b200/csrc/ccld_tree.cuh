// Tree communicators (Sec. 4.2.1): SendCount / RecvCount and their update frequencies are comparable between members of
// one tree layer only. The window decision names a slowed communicator's communication root from the rate columns of
// the selected round; for a tree that choice is redone here, layer by layer. Included by ccld_kernels.cuh.
#pragma once

namespace ccld {

struct TreeRef { u32 c, pad; const u32* head; };   // communicator index; head[p] = lowest position of p's layer

struct OpMaxU32 { __device__ u32 operator()(u32 a, u32 b) const { return a > b ? a : b; } static __device__ u32 identity() { return 0; } };

constexpr int TREE_THREADS = 256;

// One CTA per (tree communicator, window), after k_window_decide. The change count of a member is the larger of its two
// rate columns in the selected round; the root is the member with the most changes above its layer's fewest (equal
// excesses: the lowest position). If no layer disagrees with itself the rates name nobody and the member with the
// longest duration stands in, as it does for a window without rate columns.
__global__ void __launch_bounds__(TREE_THREADS) k_tree_root_comm(const WinDesc* __restrict__ wd, const TreeRef* __restrict__ trees, Registry R) {
  __shared__ u32 s_ch[CCLD_MAX_COMM_SIZE];
  __shared__ u32 s_red[32];
  const TreeRef T = trees[blockIdx.x];
  const WinDesc& D = wd[blockIdx.y];
  const RangeRow row = D.ranges[T.c];
  if (row.n_seq == 0) return;
  ccld_comm_verdict* v = D.comm_rows + row.row_idx;
  if (!v->slow_detected || v->sel_seq == NONE) return;          // the same answer in every thread
  const u32 n = R.comm_n[T.c], k = v->sel_seq - row.seq_lo;
  const u32* mem = R.members + R.comm_moff[T.c];
  for (u32 p = threadIdx.x; p < n; p += TREE_THREADS) {
    const u32 idx = D.perm[perm_at(row, k, p)];
    u32 ch = 0;
    if (D.send_chg != nullptr && idx != NONE) { const u32 a = D.send_chg[idx], b = D.recv_chg[idx]; ch = a > b ? a : b; }
    s_ch[p] = ch;
  }
  __syncthreads();
  // the lowest position of a layer walks it: fewest changes, most changes and the first member that shows those
  u32 gap = 0, cand = NONE;
  for (u32 p = threadIdx.x; p < n; p += TREE_THREADS) {
    if (T.head[p] != p) continue;
    u32 lmn = s_ch[p], lmx = lmn, at = p;
    for (u32 x = p + 1; x < n; ++x) {
      if (T.head[x] != p) continue;
      const u32 c = s_ch[x];
      if (c > lmx) { lmx = c; at = x; }
      lmn = c < lmn ? c : lmn;
    }
    const u32 g = lmx - lmn;
    if (g > gap || (g == gap && g > 0 && at < cand)) { gap = g; cand = at; }
  }
  const u32 best = block_reduce(gap, OpMaxU32(), s_red);
  if (gap != best || best == 0) cand = NONE;
  const u32 root = block_reduce(cand, OpMinU32(), s_red);
  if (threadIdx.x == 0) {
    if (root != NONE) { v->root_comm = mem[root]; v->rate_source = 0; }
    else { v->root_comm = D.gu32[(u64)GU_RANK_TMAX * D.n_groups + row.group0 + k]; v->rate_source = 1; }
  }
}

}  // namespace ccld
