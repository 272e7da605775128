// ccld_ring_locate_static: the hang decision tree over one ring, for callers that may not allocate.
//
// Who needs this: code that runs where device allocation is off the table - a watchdog thread that
// must diagnose a job whose memory is exhausted or whose allocator is wedged behind the very hang
// being diagnosed, a plugin that lives inside another process (a CCL profiler hook, a framework
// extension) and is forbidden to touch that process's memory pool, or a tight monitoring loop where
// an allocation could synchronize the device. Everything this entry point needs beyond the caller's
// own buffers sits in one fixed array that is part of the library's device image.
//
// What "allocates nothing" covers: the entry point itself never calls cudaMalloc, cudaFree or an
// allocating library routine. The CUDA runtime, however, creates a device's primary context and loads
// this library's device image (array and kernel) lazily, on the first call that names that device, and
// that one-time step takes device memory and can fail when none is left. So the first call on a
// device is the set-up call: make it once at start-up, while memory is still available (any small
// ring will do), and only the calls after it are free of allocation. It is an ordinary host function
// (runtime calls, snprintf): call it from a thread, never from a signal handler.
//
// The scratch array is shared by every call on a device and keeps whatever the last call left in it.
// The kernel overwrites every byte it later reads, so stale contents are harmless, but two calls
// whose kernels overlap on the GPU (different streams, different host threads) race on it.
#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <cuda_runtime.h>

#include "../../include/ccld.h"

namespace {

typedef uint64_t u64;
typedef uint32_t u32;
typedef uint8_t u8;

constexpr u32 NONE32 = 0xFFFFFFFFu;
constexpr u32 MAX_N = CCLD_STATIC_MAX_MEMBERS;

// Scratch layout: per-member counter totals, the root list, the result struct.
constexpr size_t OFF_TOT = 0;
constexpr size_t OFF_ROOTS = OFF_TOT + (size_t)MAX_N * 8;
constexpr size_t OFF_OUT = OFF_ROOTS + (size_t)MAX_N * 4;
constexpr size_t SCRATCH_BYTES = OFF_OUT + 256;
static_assert(SCRATCH_BYTES == CCLD_STATIC_SCRATCH_BYTES, "header and implementation disagree on the scratch size");

// Lives in every GPU's copy of the library's device image from the moment the runtime loads it there (the first call
// on that device) until exit. In host code this name is only a handle for cudaGetSymbolAddress; it is never passed
// to a kernel as if it were a device address.
static __device__ __align__(256) unsigned char g_ring_scratch[SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
// Device address of g_ring_scratch on each device, once looked up. Host threads may race to fill an entry; they all
// store the same address, and the atomic makes the publication well defined.
std::atomic<void*> g_scratch_addr[MAX_DEVICES];

template <class T, class Op>
__device__ T cta_reduce(T v, Op op, T* s_red /*[32]*/) {
  const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) { T o = __shfl_xor_sync(0xFFFFFFFFu, v, d); v = op(v, o); }
  __syncthreads();
  if (lane == 0) s_red[wid] = v;
  __syncthreads();
  T r = s_red[0];
  for (u32 q = 1; q < blockDim.x / 32; ++q) r = op(r, s_red[q]);
  return r;
}
struct AddU32 { __device__ u32 operator()(u32 a, u32 b) const { return a + b; } };
struct MinU32 { __device__ u32 operator()(u32 a, u32 b) const { return a < b ? a : b; } };
struct MinU64 { __device__ u64 operator()(u64 a, u64 b) const { return a < b ? a : b; } };

// One CTA. state[p]: bit0 member p entered the op, bit1 its record of the op is complete, bit2 it has a
// progress frame; progress[p][channel][0/1] = SendCount / RecvCount of member p (ring position order).
__global__ void __launch_bounds__(1024) k_ring_locate_static(u32 n, const u32* __restrict__ ranks, const u8* __restrict__ state,
                                                              u32 n_channels, const u32* __restrict__ progress,
                                                              unsigned char* __restrict__ scratch) {
  __shared__ u64 s_red64[32];
  __shared__ u32 s_red32[32];
  __shared__ u32 s_base;
  u64* tot = (u64*)(scratch + OFF_TOT);
  u32* roots = (u32*)(scratch + OFF_ROOTS);
  ccld_hang_verdict* out = (ccld_hang_verdict*)(scratch + OFF_OUT);

  u32 n_ne = 0, n_ok = 0, n_missing = 0; u64 mn = ~0ull;
  for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
    const u8 st = state[p];
    n_ne += !(st & 1); n_ok += (st & 2) ? 1u : 0u;
    u64 t = 0;
    if (!(st & 4)) ++n_missing;
    else for (u32 ch = 0; ch < n_channels; ++ch) t += (u64)progress[((u64)p * n_channels + ch) * 2] + progress[((u64)p * n_channels + ch) * 2 + 1];
    tot[p] = t;                                   // every entry below n is rewritten before it is read
    mn = t < mn ? t : mn;
  }
  n_ne = cta_reduce(n_ne, AddU32(), s_red32);
  n_ok = cta_reduce(n_ok, AddU32(), s_red32);
  n_missing = cta_reduce(n_missing, AddU32(), s_red32);
  mn = cta_reduce(mn, MinU64(), s_red64);
  __syncthreads();
  const u32 cls = n_ne > 0 ? 1u : (n_ok > 0 ? 2u : 3u);
  u32 n_roots = 0, stuck = 0; u64 min_total = 0;
  if (cls == 3) {
    u32 up = NONE32, any = NONE32;
    for (u32 p = threadIdx.x; p < n; p += blockDim.x) {
      if (tot[p] != mn) continue;
      any = p < any ? p : any;
      if (tot[(p + n - 1) % n] > mn) up = p < up ? p : up;
    }
    up = cta_reduce(up, MinU32(), s_red32);
    any = cta_reduce(any, MinU32(), s_red32);
    const u32 root = up != NONE32 ? up : any;
    n_roots = 1; min_total = mn;
    if (threadIdx.x == 0) {
      roots[0] = ranks[root];
      if ((state[root] & 4) && n_channels > 0) {
        u32 s = NONE32;
        for (u32 ch = 0; ch < n_channels; ++ch) { const u32 r = progress[((u64)root * n_channels + ch) * 2 + 1]; s = r < s ? r : s; }
        stuck = s;
      }
    }
  } else {
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (u32 p0 = 0; p0 < n; p0 += blockDim.x) {
      const u32 p = p0 + threadIdx.x;
      const bool sel = p < n && (cls == 1 ? !(state[p] & 1) : (state[p] & 2) != 0);
      const u32 bal = __ballot_sync(0xFFFFFFFFu, sel);
      const u32 lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
      __syncthreads();
      if (lane == 0) s_red32[wid] = __popc(bal);
      __syncthreads();
      u32 off = s_base;
      for (u32 q = 0; q < wid; ++q) off += s_red32[q];
      off += __popc(bal & ((1u << lane) - 1));
      if (sel) roots[off] = ranks[p];
      __syncthreads();
      if (threadIdx.x == 0) { u32 t = 0; for (u32 q = 0; q < blockDim.x / 32; ++q) t += s_red32[q]; s_base += t; }
      __syncthreads();
    }
    n_roots = s_base;
  }
  if (threadIdx.x == 0) {
    ccld_hang_verdict v;
    v.cls = cls; v.n_roots_total = n_roots; v.n_not_entered = n_ne; v.n_hung = n - n_ok; v.n_not_hung = n_ok;
    v.n_missing_frames = cls == 3 ? n_missing : 0; v.stuck_step = stuck; v.n_members = n; v.min_total = min_total;
    v.roots = nullptr; v.roots_cap = 0;
    *out = v;
  }
}

int say(char* err, uint32_t cap, int code, const char* msg) {
  if (err && cap) std::snprintf(err, cap, "%s", msg);
  return code;
}

}  // namespace

extern "C" int ccld_ring_locate_static(int device, void* cuda_stream, uint32_t n_members, const uint32_t* ranks, const uint8_t* state,
                                       uint32_t n_channels, const uint32_t* progress, ccld_hang_verdict* out, char* err, uint32_t err_cap) {
  if (!out || !ranks || !state || n_members == 0) return say(err, err_cap, CCLD_ERR_ARG, "null pointer or empty ring");
  if (n_members > MAX_N) return say(err, err_cap, CCLD_ERR_CAPACITY, "ring larger than CCLD_STATIC_MAX_MEMBERS: the fixed scratch cannot hold it");
  if (n_channels > 0 && !progress) return say(err, err_cap, CCLD_ERR_ARG, "n_channels > 0 but no progress table");
  if (device < 0 || device >= MAX_DEVICES) return say(err, err_cap, CCLD_ERR_ARG, "device ordinal out of range");
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return say(err, err_cap, CCLD_ERR_CUDA, "cudaGetDevice failed");
  if (cudaSetDevice(device) != cudaSuccess) return say(err, err_cap, CCLD_ERR_CUDA, "cudaSetDevice failed");
  int rc = CCLD_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // set-up, once per device and with that device current: ask the runtime where the array lives there
  if (g_scratch_addr[device].load(std::memory_order_acquire) == nullptr) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_ring_scratch);
    if (e != cudaSuccess || p == nullptr) {
      rc = say(err, err_cap, e == cudaErrorMemoryAllocation ? CCLD_ERR_NOMEM : CCLD_ERR_CUDA, cudaGetErrorString(e)); goto done;
    }
    g_scratch_addr[device].store(p, std::memory_order_release);
  }
  {
    unsigned char* scratch = (unsigned char*)g_scratch_addr[device].load(std::memory_order_acquire);
    k_ring_locate_static<<<1, 1024, 0, st>>>(n_members, ranks, state, n_channels, progress, scratch);
    cudaError_t e = cudaGetLastError();
    ccld_hang_verdict v;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&v, scratch + OFF_OUT, sizeof v, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { rc = say(err, err_cap, CCLD_ERR_CUDA, cudaGetErrorString(e)); goto done; }
    uint32_t* roots = out->roots; const uint32_t cap = roots ? out->roots_cap : 0;
    *out = v; out->roots = roots; out->roots_cap = cap;
    uint32_t n_copy = v.n_roots_total < n_members ? v.n_roots_total : n_members;
    if (n_copy > cap) n_copy = cap;
    if (n_copy) {
      e = cudaMemcpyAsync(roots, scratch + OFF_ROOTS, (size_t)n_copy * 4, cudaMemcpyDeviceToHost, st);
      if (e == cudaSuccess) e = cudaStreamSynchronize(st);
      if (e != cudaSuccess) rc = say(err, err_cap, CCLD_ERR_CUDA, cudaGetErrorString(e));
    }
  }
done:
  if (prev >= 0 && prev != device) cudaSetDevice(prev);
  return rc;
}
