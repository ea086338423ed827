// dslide_bucket_sort_static: group neuron ids by bucket code (one hash table) without allocating.
//
// Some callers may not allocate device memory when they reach this library: code that runs inside
// a memory pool it does not own, a serving loop that has promised its operator a fixed footprint,
// a plug-in that is handed buffers by its host application and nothing else.  For them this one
// entry point keeps every byte of its work space in a file-scope __device__ array that is part of
// the loaded library image, so the call makes no cudaMalloc, no cudaFree and no library call that
// allocates.  The price: every GPU that loads libdslide.so holds the array (2 MiB) until the
// process exits, the problem size is capped, and all calls share the one array.
//
// The work is the table build's stable sort (ids grouped by code, ascending inside a group) done by a
// single thread block: a least-significant-digit radix sort with 9-bit digits whose per-warp digit
// counters live in shared memory and whose intermediate (key, id) pairs live in the static array.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dslide.h"

namespace {

constexpr int SS_THREADS = 512;
constexpr int SS_WARPS = SS_THREADS / 32;
constexpr int SS_WIDTH = 9;
constexpr int SS_RADIX = 1 << SS_WIDTH;

// Work space: [max n] keys followed by [max n] ids.  Only host code needs its device address
// (cudaGetSymbolAddress below); the name itself is not a device pointer on the host side.
static __device__ __align__(256) unsigned char g_static_scratch[(size_t)DSLIDE_STATIC_SORT_MAX_N * 8];

__global__ void __launch_bounds__(SS_THREADS)
k_bucket_sort_static(const uint32_t* __restrict__ codes, int n, int bits, int32_t* bucket_off, int32_t* bucket_ids,
                     uint32_t* tmp_keys, int32_t* tmp_vals) {
  __shared__ int offs[SS_WARPS][SS_RADIX];
  __shared__ int sh[SS_WARPS + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nb = 1 << bits;
  const uint32_t cmask = (uint32_t)nb - 1u;

  // ---- bucket offsets: clear (the output array may hold anything), count, running sum ----
  for (int i = tid; i <= nb; i += SS_THREADS) bucket_off[i] = 0;
  __syncthreads();
  for (int i = tid; i < n; i += SS_THREADS) atomicAdd(&bucket_off[(codes[i] & cmask) + 1], 1);
  __syncthreads();
  {
    const int total = nb + 1;
    const int chunk = (total + SS_THREADS - 1) / SS_THREADS;
    const int beg = min(total, tid * chunk), end = min(total, beg + chunk);
    int sum = 0;
    for (int i = beg; i < end; ++i) sum += bucket_off[i];
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += v;
    }
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < SS_WARPS; ++w) { int c = sh[w]; sh[w] = run; run += c; }
    }
    __syncthreads();
    int run = incl - sum + sh[warp];
    for (int i = beg; i < end; ++i) { run += bucket_off[i]; bucket_off[i] = run; }
  }
  __syncthreads();

  // ---- stable radix sort of the ids by code; each warp owns a contiguous run of the input ----
  const int passes = (bits + SS_WIDTH - 1) / SS_WIDTH;
  const int width0 = (bits + passes - 1) / passes;
  int sub = (n + SS_WARPS - 1) / SS_WARPS;
  sub = (sub + 31) & ~31;
  const int wbeg = min(n, warp * sub), wend = min(n, wbeg + sub);
  for (int pass = 0; pass < passes; ++pass) {
    const int shift = pass * width0;
    const int width = min(width0, bits - shift);
    const int radix = 1 << width;
    const bool first = pass == 0, last = pass == passes - 1;
    const uint32_t* kin = first ? codes : tmp_keys;

    for (int d = lane; d < radix; d += 32) offs[warp][d] = 0;
    __syncwarp();
    for (int i = wbeg + lane; i < wend; i += 32) atomicAdd(&offs[warp][((kin[i] & cmask) >> shift) & (radix - 1)], 1);
    __syncthreads();
    // where the run of digit d of warp w starts: all smaller digits, then the same digit in earlier warps
    int tot = 0;
    if (tid < radix)
      for (int w = 0; w < SS_WARPS; ++w) tot += offs[w][tid];
    int incl = tot;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += v;
    }
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < SS_WARPS; ++w) { int c = sh[w]; sh[w] = run; run += c; }
    }
    __syncthreads();
    if (tid < radix) {
      int run = incl - tot + sh[warp];
      for (int w = 0; w < SS_WARPS; ++w) { int c = offs[w][tid]; offs[w][tid] = run; run += c; }
    }
    __syncthreads();
    for (int i0 = wbeg; i0 < wend; i0 += 32) {
      const int i = i0 + lane;
      const bool live = i < wend;
      const uint32_t key = live ? (kin[i] & cmask) : 0u;
      const int digit = live ? (int)((key >> shift) & (radix - 1)) : radix + lane;
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      const int rank = __popc(peers & ((1u << lane) - 1u));
      int base = 0;
      if (live) base = offs[warp][digit];
      __syncwarp();
      if (live && rank == 0) offs[warp][digit] = base + __popc(peers);
      __syncwarp();
      if (live) {
        const int dst = base + rank;
        const int id = first ? i : tmp_vals[i];
        if (last) bucket_ids[dst] = id;
        else { tmp_keys[dst] = key; tmp_vals[dst] = id; }
      }
    }
    __syncthreads();
  }
}

// Device address of the static work space, looked up once per device.
constexpr int SS_MAX_DEVICES = 64;
unsigned char* g_scratch_addr[SS_MAX_DEVICES];

}  // namespace

extern "C" dslide_status dslide_bucket_sort_static(const uint32_t* codes, int32_t n, int32_t bits,
                                                   int32_t* bucket_off, int32_t* bucket_ids, void* stream) {
  if (!codes || !bucket_off || !bucket_ids) return DSLIDE_ERR_INVALID_ARG;
  if (n < 0 || n > DSLIDE_STATIC_SORT_MAX_N) return DSLIDE_ERR_OVERFLOW;
  if (bits < 1 || bits > DSLIDE_STATIC_SORT_MAX_BITS) return DSLIDE_ERR_OVERFLOW;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= SS_MAX_DEVICES) return DSLIDE_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    // first call on this device: ask the runtime where the array lives on the current device
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return DSLIDE_ERR_CUDA; }
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  uint32_t* tmp_keys = reinterpret_cast<uint32_t*>(g_scratch_addr[dev]);
  int32_t* tmp_vals = reinterpret_cast<int32_t*>(g_scratch_addr[dev] + (size_t)DSLIDE_STATIC_SORT_MAX_N * 4);
  k_bucket_sort_static<<<1, SS_THREADS, 0, (cudaStream_t)stream>>>(codes, n, bits, bucket_off, bucket_ids, tmp_keys,
                                                                  tmp_vals);
  return cudaGetLastError() == cudaSuccess ? DSLIDE_OK : DSLIDE_ERR_CUDA;
}
