// Operation Type Set consistency of one op (Sec. 4.1.2: algorithm, protocol, data size and operation name are constant
// during a communication; Sec. 4.2.2: inconsistent operations are what leaf H2 of the hang tree points at). One CTA:
// the most frequent (op, bytes, algo, proto) among the members that reported the op - ties go to the tuple whose
// first holder stands earliest in the ring - and the members that carry another tuple, in ring order.
#pragma once
#include "ccld_kernels.cuh"

namespace ccld {

struct OpsetArgs {
  u32 c, seq;
  const u8 *algo, *proto;        // per record, may both be null (then 0)
  u64* key_hi; u32* key_lo;      // [n] scratch: bytes, op | algo << 8 | proto << 16 | present << 31
  u32* ranks; u32 ranks_cap;     // device list of the deviating ranks
  ccld_opset_verdict* out;       // device copy (pointer fields unused)
};

__global__ void __launch_bounds__(1024) k_opset_check(const WinDesc* __restrict__ wd, Registry R, OpsetArgs A) {
  __shared__ u64 s_red64[32];
  __shared__ u32 s_red32[32];
  __shared__ u32 s_base;
  const WinDesc& D = wd[0];
  const u32 c = A.c, n = R.comm_n[c];
  const u32* mem = R.members + R.comm_moff[c];
  const RangeRow row = D.ranges[c];
  const bool in_range = row.n_seq > 0 && A.seq >= row.seq_lo && A.seq - row.seq_lo < row.n_seq;
  u32 n_present = 0;
  for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
    const u32 idx = in_range ? D.perm[perm_at(row, A.seq - row.seq_lo, p)] : NONE;
    u64 hi = 0; u32 lo = 0;
    if (idx != NONE) {
      hi = D.bytes[idx];
      lo = (u32)D.op[idx] | (A.algo ? (u32)A.algo[idx] << 8 : 0u) | (A.proto ? (u32)A.proto[idx] << 16 : 0u) | 0x80000000u;
      ++n_present;
    }
    A.key_hi[p] = hi; A.key_lo[p] = lo;
  }
  n_present = block_reduce(n_present, OpAddU32(), s_red32);
  __syncthreads();
  // how many members share each member's tuple; the best is the largest count, then the lowest position
  u64 best = 0;
  for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
    const u64 hi = A.key_hi[p]; const u32 lo = A.key_lo[p];
    if (!(lo & 0x80000000u)) continue;
    u32 cnt = 0;
    for (u32 q = 0; q < n; ++q) cnt += (A.key_lo[q] == lo && A.key_hi[q] == hi) ? 1u : 0u;
    const u64 k = ((u64)cnt << 32) | (u64)(NONE - p);
    best = k > best ? k : best;
  }
  best = block_reduce(best, OpMaxU64(), s_red64);
  __syncthreads();
  const u32 maj_cnt = (u32)(best >> 32), maj_p = maj_cnt ? NONE - (u32)best : 0u;
  const u64 m_hi = maj_cnt ? A.key_hi[maj_p] : 0; const u32 m_lo = maj_cnt ? A.key_lo[maj_p] : 0;
  // ordered compaction of the deviating members
  if (threadIdx.x == 0) s_base = 0;
  __syncthreads();
  for (u32 p0 = 0; p0 < n; p0 += blockDim.x) {
    const u32 p = p0 + threadIdx.x;
    const bool sel = p < n && (A.key_lo[p] & 0x80000000u) && (A.key_lo[p] != m_lo || A.key_hi[p] != m_hi);
    const u32 bal = __ballot_sync(0xFFFFFFFFu, sel);
    const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) s_red32[wid] = __popc(bal);
    __syncthreads();
    u32 off = s_base;
    for (u32 q = 0; q < wid; ++q) off += s_red32[q];
    off += __popc(bal & ((1u << lane) - 1));
    if (sel && off < A.ranks_cap) A.ranks[off] = mem[p];
    __syncthreads();
    if (threadIdx.x == 0) { u32 tot = 0; for (u32 q = 0; q < blockDim.x / 32; ++q) tot += s_red32[q]; s_base += tot; }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ccld_opset_verdict v;
    v.n_members = n; v.n_present = n_present; v.n_deviating_total = s_base; v.majority_count = maj_cnt;
    v.op = (u8)(m_lo & 0xFF); v.algo = (u8)((m_lo >> 8) & 0xFF); v.proto = (u8)((m_lo >> 16) & 0xFF); v.pad = 0;
    v.bytes = m_hi; v.ranks = nullptr; v.ranks_cap = 0;
    *A.out = v;
  }
}

}  // namespace ccld
