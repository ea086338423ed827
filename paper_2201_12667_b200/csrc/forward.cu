// Per-sample forward kernel of the SLIDE step: one thread block per sample runs
//   hidden layer (Section 3.6, feed forward of the first type: sparse input)
//   -> L bucket codes of the hidden activation (SimHash or DWTA, Section 4.1)
//   -> bucket lookup, union over the tables plus the labels (Section 2.1, Fig. 1)
//   -> logits over the active set only (feed forward of the second type)
//   -> softmax, loss and errors over that ragged set (Algorithm 1 "Compute Errors")
//   -> error back-propagated to the hidden layer (Section 2.1, back-propagation stage)
// and hands the touched rows of W2 and W1 to the update kernel.
// The same kernel in predict mode stops after the logits and selects the top k.
//
// Every phase is a short chain of memory rounds, so each round puts as much in flight as it can:
// the rows of W1 of a chunk of nonzeros arrive by one bulk copy each (cp.async.bulk, completion on an
// mbarrier) and are then summed in the stored order; the L bucket offsets are fetched in one round and
// all bucket entries in a second; the active rows of W2 are copied the same way into the shared memory
// the dedup work space no longer needs, and serve both the logits and the back-propagated error (in
// one pass when the set is larger than that space).  Optional steps of the selection: densification
// of all-zero DWTA bins of the query (Section 4.1) and the sampling budget of Section 3.7.
#include "common.cuh"

namespace dslide {

constexpr int FWD_THREADS = 256;
constexpr int FWD_WARPS = FWD_THREADS / 32;
constexpr int MAX_KPT = 4;        // hidden units per thread: H <= 4 * 256
constexpr int ACT_SM = 1024;      // active ids and logits are mirrored in shared memory when the set is this small
constexpr int HID_MIN_BYTES = 64 * 1024;   // staging space for the hidden layer's rows of W1
constexpr int RANK_MAX = 1024;    // candidate sets up to this size are put in order by counting, larger ones by a bitonic sort
constexpr int SORT_SMALL = 1024;  // candidate sets up to this size are sorted rather than run through the bitmap
constexpr unsigned FULLM = 0xffffffffu;

struct FwdParams {
  const float *W1, *b1, *W2;
  const int32_t *hash_idx, *hash_sign, *bucket_off, *bucket_ids;
  const int32_t *row_ptr, *col_idx;
  const float* vals;
  const int32_t *label_ptr, *labels;
  float *h, *dh, *loss;
  uint32_t* codes;
  int32_t *act_cnt, *act_ids;
  float *act_z, *act_p, *act_g;
  uint32_t *mask1, *mask2;
  int2 *ovf1, *ovf2;
  const int32_t* hotmap1;   // rows of W1 with a line of the coefficient table
  float* hotcoef1;
  int bstride;              // samples per line of that table
  RowHdr *hdr1, *hdr2;
  int2 *own1, *own2;
  int32_t *hot_rows, *med_rows;
  DevState* st;
  int32_t* out_ids;
  float* out_scores;
  long long nb;
  int B, D, H, N, K, L, KL, family, lg_bin, fn_len, cap;
  int act_stride, Wd, dense, dedup_mode, max_labels, sort_cap, topk, parity;
  int stage_bytes;     // bytes of the staging region (it starts at off_dedup and overlays the dedup work space)
  int hid_rows;        // rows of W1 staged per chunk of the hidden layer
  int budget;          // Section 3.7: active neurons kept per sample, labels included (0 = no budget)
  int budget_fill;     // Section 3.7: a set below the budget is topped up with uniform draws
  unsigned long long tcount;   // steps taken so far (the reservoir's draws are numbered by step, sample and candidate)
  int densify;         // DWTA: all-zero bins of the query borrow another bin's position
  unsigned long long seed, rcount;   // for the probe sequence of the densification: the model's seed, rebuilds so far
  int hash_sm_off;     // where in the staging region the hash functions' index tables are mirrored (-1: read from global memory)
  int hash_sm_bytes;
  int sort_small;      // candidate sets up to this size are deduplicated by sorting even when a bitmap is available
  // LSH-sampled hidden layer (L1 > 0): projections over the input coordinates, tables over the hidden neurons
  const int8_t* proj1;
  const int32_t *bucket1_off, *bucket1_ids;
  uint32_t *codes1, *hmask, *cmask1;
  int K1, L1, KL1, cap1, Hw, off_h1;
  int inputs_ready;    // the batch arrays were complete before the launch: they may be read before griddep_wait()
  int off_dh, off_code, off_part, off_misc, off_lab, off_tbase, off_tbeg, off_topk, off_ids, off_z, off_col, off_val,
      off_dedup;
};

__device__ __forceinline__ void set_status(DevState* st, int code) { atomicCAS(&st->status, 0, code); }

// ---- bulk copy (global -> shared) with completion on an mbarrier ------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// 16-byte asynchronous copy global -> shared (through L2 only), and the wait for all of a thread's copies
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Waits for the phase with the given parity; gives up after a bounded number of polls (false).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t a = smem_u32(bar);
  for (int it = 0; it < (1 << 22); ++it) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(a), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}

// The touch that takes a row past ROW_SLOTS touching samples enters the row in the list of rows that a warp of
// the update kernel sums from slots and mask; the touch that takes it past HOT_T enters it in the list of rows
// summed in slices.  The row's count word is marked so that the update kernel knows where the row is listed.
__device__ __forceinline__ void list_row(const FwdParams& p, uint32_t* cnt, int code, unsigned nth) {
  if (nth == (unsigned)ROW_SLOTS) {
    const unsigned at = atomicAdd(&p.st->n_med[p.parity], 1u);
    if (at < (unsigned)MED_CAP) {
      p.med_rows[at] = code;
      atomicOr(cnt, CNT_MED);
    }
  }
  if (nth == (unsigned)HOT_T) {
    const unsigned at = atomicAdd(&p.st->n_hot[p.parity], 1u);
    if (at < (unsigned)HOT_CAP) {
      p.hot_rows[at] = code;
      atomicOr(cnt, CNT_HOT);
    }
  }
}

// Handing a touched row to the update kernel, once the row's touch counter has answered (nth = touches before this
// one).  touch_mark: the (sample, coefficient) pair goes into the row's slot nth, or, past the slots, the sample's bit
// into the row's mask (and, up to PAIR_T touches, the pair into the side array); the touch that fills the slots or
// reaches HOT_T lists the row (list_row: an atomic whose answer is needed, so callers on the critical path put it
// off to the end of the kernel).  own_reserve / own_store: the first toucher enters (row, its own sample) in the list
// of distinct rows, so that the update kernel can fetch that sample's row at once; positions are handed out per
// warp by one atomic, asked for by own_reserve and used by own_store (callers put other work in between, so that
// no warp waits for the answer).  All three are called by whole warps; `live` tells whether this thread has a touch.
template <bool LIST = true>      // LIST = false: the caller lists the row (list_row) itself, later
__device__ __forceinline__ void touch_mark(const FwdParams& p, bool live, RowHdr* hd, uint32_t* maskrow, int2* ovfrow, int code,
                                           unsigned nth, int s, float coef) {
  if (!live) return;
  if (nth < (unsigned)ROW_SLOTS) hd->slot[nth] = make_int2(s, __float_as_int(coef));
  else {
    atomicOr(maskrow + (s >> 5), 1u << (s & 31));
    // up to PAIR_T touches keep their pair as well, so that a row with that many is summed without any search
    if (nth < (unsigned)PAIR_T) ovfrow[nth] = make_int2(s, __float_as_int(coef));
  }
  if (LIST) list_row(p, &hd->cnt, code, nth);
}
__device__ __forceinline__ unsigned own_reserve(bool first, unsigned int* n_own) {
  const unsigned fm = __ballot_sync(FULLM, first);
  unsigned base = 0;
  if (fm && (threadIdx.x & 31) == 0) base = atomicAdd(n_own, (unsigned)__popc(fm));
  return base;                                   // valid in lane 0
}
__device__ __forceinline__ void own_store(bool first, unsigned base, int2* own, int row, int s) {
  const int lane = threadIdx.x & 31;
  const unsigned fm = __ballot_sync(FULLM, first);
  if (!fm) return;
  base = __shfl_sync(FULLM, base, 0);
  if (first) own[base + __popc(fm & ((1u << lane) - 1u))] = make_int2(row, s);
}
__device__ __forceinline__ void finish_touch(const FwdParams& p, bool live, RowHdr* hd, uint32_t* maskrow, int2* ovfrow, int2* own,
                                             unsigned int* n_own, int row, int code, unsigned nth, int s, float coef) {
  touch_mark(p, live, hd, maskrow, ovfrow, code, nth, s, coef);
  const bool first = live && nth == 0u;
  const unsigned base = own_reserve(first, n_own);
  own_store(first, base, own, row, s);
}

// Maximum / sum over the lanes of a warp in a fixed order (same value in every lane).
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(FULLM, v, d));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(FULLM, v, d);
  return v;
}

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
// sh needs FWD_WARPS + 1 ints.  Ends with a barrier, so sh may be reused afterwards.
__device__ __forceinline__ int block_excl_scan(int v, int* sh, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int n = __shfl_up_sync(FULLM, incl, d);
    if (lane >= d) incl += n;
  }
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int w = 0; w < FWD_WARPS; ++w) { int c = sh[w]; sh[w] = run; run += c; }
    sh[FWD_WARPS] = run;
  }
  __syncthreads();
  int res = incl - v + sh[warp];
  *total = sh[FWD_WARPS];
  __syncthreads();
  return res;
}

// Block-wide max / sum in a fixed order (same value in every thread).  sh: FWD_WARPS floats.
__device__ __forceinline__ float block_max(float v, float* sh) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(FULLM, v, d));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int w = 1; w < FWD_WARPS; ++w) r = fmaxf(r, sh[w]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float block_sum(float v, float* sh) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(FULLM, v, d);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int w = 1; w < FWD_WARPS; ++w) r += sh[w];
  __syncthreads();
  return r;
}

__device__ __forceinline__ bool topk_better(float za, int ia, float zb, int ib) {
  return za > zb || (za == zb && ia < ib);
}

// Puts n <= PER * FWD_THREADS values in ascending order by counting: the place of a value is the number of values
// before it (by value, then by position).  src and dst are in shared memory; thread t owns the values t, t +
// FWD_THREADS, ...; threads without a value skip the counting loop.
// PACKED: src holds (value << RANK_BITS | position), padded with 0xffffffff to a multiple of four -- all distinct,
// so one comparison per pair decides; dst receives the values alone.
constexpr int RANK_BITS = 10;
template <int PER, bool PACKED>
__device__ __forceinline__ void rank_sort(const uint32_t* src, uint32_t* dst, int n) {
  const int tid = threadIdx.x;
  if (tid >= n) return;
  uint32_t v[PER];
  int pos[PER];
#pragma unroll
  for (int u = 0; u < PER; ++u) {
    const int i = tid + u * FWD_THREADS;
    v[u] = i < n ? src[i] : 0xffffffffu;
    pos[u] = 0;
  }
  if (PACKED) {
    const uint4* src4 = reinterpret_cast<const uint4*>(src);
    const int n4 = (n + 3) >> 2;
#pragma unroll 2
    for (int k = 0; k < n4; ++k) {
      const uint4 a = src4[k];
#pragma unroll
      for (int u = 0; u < PER; ++u)
        pos[u] += (a.x < v[u] ? 1 : 0) + (a.y < v[u] ? 1 : 0) + (a.z < v[u] ? 1 : 0) + (a.w < v[u] ? 1 : 0);
    }
#pragma unroll
    for (int u = 0; u < PER; ++u)
      if (tid + u * FWD_THREADS < n) dst[pos[u]] = v[u] >> RANK_BITS;
  } else {
#pragma unroll 4
    for (int k = 0; k < n; ++k) {
      const uint32_t a = src[k];
#pragma unroll
      for (int u = 0; u < PER; ++u) pos[u] += (a < v[u] || (a == v[u] && k < tid + u * FWD_THREADS)) ? 1 : 0;
    }
#pragma unroll
    for (int u = 0; u < PER; ++u)
      if (tid + u * FWD_THREADS < n) dst[pos[u]] = v[u];
  }
}

// Section 3.7, the fill option: a set below the budget is topped up with neurons drawn one after the other,
// id_k = rng(seed, RNG_FILL, steps taken, sample * 2^32 + k) mod N; a draw already in the set (retrieved, label, or
// drawn before) is passed over; drawing stops when the set has min(budget, N) members or after 2 * missing + 64
// draws.  All draws are evaluated at once: a shared-memory hash set records the first draw of every id, a search in
// the (ascending) set tells which ids are new, and the running count in draw order says which of them still fit.
// The accepted ids are put in order and merged with the set.  Returns the new count.
__device__ __forceinline__ int fill_work_bytes(int need) {
  const int D = 2 * need + 64;
  int ts = 64;
  while (ts < 2 * D) ts <<= 1;
  return 4 * D + ((D + 3) & ~3) + 8 * ts + 8 * need;       // draws, flags, hash set (ids, first draws), accepted ids twice
}
__device__ __noinline__ int budget_fill(int budget, int N, uint64_t seed, uint64_t tcount, int s, int32_t* ids, int* sh_ids,
                                        int na, unsigned char* work, int work_bytes, int* sh_scan, DevState* st) {
  const int tid = threadIdx.x;
  const int target = min(budget, N);
  if (na >= target) return na;
  const int need = target - na;
  const int D = 2 * need + 64;
  int ts = 64;
  while (ts < 2 * D) ts <<= 1;
  if (fill_work_bytes(need) + 4 * target > work_bytes) {     // cannot happen with the sizes checked at start-up
    if (tid == 0) set_status(st, DSLIDE_ERR_OVERFLOW);
    return na;
  }
  int* draw = reinterpret_cast<int*>(work);                 // [D]
  unsigned char* okf = reinterpret_cast<unsigned char*>(draw + D);       // [D]
  int* keys = reinterpret_cast<int*>(okf + ((D + 3) & ~3)); // [ts] ids seen, -1 = empty
  int* mink = keys + ts;                                    // [ts] the first draw of that id
  int* F = mink + ts;                                       // [need] accepted ids in draw order
  int* Fs = F + need;                                       // [need] ascending
  int* out = Fs + need;                                     // [target]
  const int lg = 31 - __clz(ts);
  for (int h = tid; h < ts; h += FWD_THREADS) { keys[h] = -1; mink[h] = 0x7fffffff; }
  for (int k = tid; k < D; k += FWD_THREADS)
    draw[k] = (int)(ctr_rng(seed, RNG_FILL, tcount, ((uint64_t)(uint32_t)s << 32) + (uint64_t)k) % (uint64_t)N);
  __syncthreads();
  for (int k = tid; k < D; k += FWD_THREADS) {
    const int id = draw[k];
    unsigned h = ((unsigned)id * 2654435761u) >> (32 - lg);
    for (int it = 0; it < ts; ++it) {
      const int prev = atomicCAS(&keys[h], -1, id);
      if (prev == -1 || prev == id) { atomicMin(&mink[h], k); break; }
      h = (h + 1) & (unsigned)(ts - 1);
    }
  }
  __syncthreads();
  for (int k = tid; k < D; k += FWD_THREADS) {
    const int id = draw[k];
    unsigned h = ((unsigned)id * 2654435761u) >> (32 - lg);
    bool first = false;
    for (int it = 0; it < ts; ++it) {
      if (keys[h] == id) { first = mink[h] == k; break; }
      h = (h + 1) & (unsigned)(ts - 1);
    }
    int lo = 0, hi = na;                                    // is the id in the set already?
    while (lo < hi) { const int mid = (lo + hi) >> 1; const int v = mid < ACT_SM ? sh_ids[mid] : ids[mid]; if (v < id) lo = mid + 1; else hi = mid; }
    const bool in_set = lo < na && (lo < ACT_SM ? sh_ids[lo] : ids[lo]) == id;
    okf[k] = (first && !in_set) ? 1 : 0;
  }
  __syncthreads();
  // running count in draw order: the first `need` new ids are accepted
  const int chunk = (D + FWD_THREADS - 1) / FWD_THREADS;
  const int k0 = min(D, tid * chunk), k1 = min(D, k0 + chunk);
  int cnt = 0;
  for (int k = k0; k < k1; ++k) cnt += okf[k];
  int total_ok = 0;
  int at = block_excl_scan(cnt, sh_scan, &total_ok);
  for (int k = k0; k < k1; ++k)
    if (okf[k]) { if (at < need) F[at] = draw[k]; ++at; }
  const int got = min(total_ok, need);
  __syncthreads();
  for (int j = tid; j < got; j += FWD_THREADS) {            // ascending order by counting (the ids are distinct)
    const int v = F[j];
    int r = 0;
    for (int q = 0; q < got; ++q) r += F[q] < v ? 1 : 0;
    Fs[r] = v;
  }
  __syncthreads();
  for (int i = tid; i < na; i += FWD_THREADS) {             // merge: each element lands after the smaller ones of both lists
    const int v = i < ACT_SM ? sh_ids[i] : ids[i];
    int lo = 0, hi = got;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (Fs[mid] < v) lo = mid + 1; else hi = mid; }
    out[i + lo] = v;
  }
  for (int j = tid; j < got; j += FWD_THREADS) {
    const int v = Fs[j];
    int lo = 0, hi = na;
    while (lo < hi) { const int mid = (lo + hi) >> 1; const int w = mid < ACT_SM ? sh_ids[mid] : ids[mid]; if (w < v) lo = mid + 1; else hi = mid; }
    out[j + lo] = v;
  }
  __syncthreads();
  const int total = na + got;
  for (int a = tid; a < total; a += FWD_THREADS) {
    ids[a] = out[a];
    if (a < ACT_SM) sh_ids[a] = out[a];
  }
  __syncthreads();
  return total;
}

// Section 3.7: the sample's retrieved neurons exceed the sampling budget -> reservoir sampling keeps
// m = max(0, budget - labels) of those that are not labels.  The textbook algorithm runs over the candidates in
// ascending id order: the first m fill the reservoir, candidate i >= m draws j uniform in [0, i] and replaces slot j
// when j < m.  Its outcome is fixed by the draws alone -- slot j ends with the LAST candidate that drew j, or with
// candidate j itself -- so the block evaluates all draws at once and settles every slot with a shared-memory max.
// ids[0 .. na) (ascending, mirrored in sh_ids up to ACT_SM) is rewritten with the labels and the reservoir,
// ascending; returns the new count.  work: 4 * na + 4 * m + nc + 4 * (m + labels) bytes of shared memory.
// Called by the whole block; kept out of line because most configurations never run it.
__device__ __noinline__ int budget_select(int budget, int fill, int N, uint64_t seed, uint64_t tcount, int s, int32_t* ids,
                                          int* sh_ids, int na, const int32_t* lab, int nlab, unsigned char* work,
                                          int work_bytes, int* sh_scan, DevState* st) {
  const int tid = threadIdx.x;
  int* cidx = reinterpret_cast<int*>(work);                 // [na] index among the candidates, -1 for a label
  const int chunk = (na + FWD_THREADS - 1) / FWD_THREADS;
  const int a0 = min(na, tid * chunk), a1 = min(na, a0 + chunk);
  int cnt = 0;
  for (int a = a0; a < a1; ++a) {
    const int id = a < ACT_SM ? sh_ids[a] : ids[a];
    bool isl = false;
    for (int i = 0; i < nlab; ++i) isl = isl || lab[i] == id;
    cidx[a] = isl ? -1 : 0;
    cnt += isl ? 0 : 1;
  }
  int nc = 0;
  int at = block_excl_scan(cnt, sh_scan, &nc);
  const int ny = na - nc;
  const int m = max(0, budget - ny);
  if (nc <= m)                                               // uniform over the block
    return fill ? budget_fill(budget, N, seed, tcount, s, ids, sh_ids, na, work, work_bytes, sh_scan, st) : na;
  for (int a = a0; a < a1; ++a)
    if (cidx[a] == 0) cidx[a] = at++;
  int* win = cidx + na;                                      // [m] the last candidate that drew the slot
  unsigned char* sel = reinterpret_cast<unsigned char*>(win + m);        // [nc]
  int* out = reinterpret_cast<int*>(work + (((size_t)4 * na + (size_t)4 * m + nc + 15) & ~(size_t)15));  // [m + ny]
  for (int j = tid; j < m; j += FWD_THREADS) win[j] = -1;
  for (int i = tid; i < nc; i += FWD_THREADS) sel[i] = 0;
  __syncthreads();
  for (int a = a0; a < a1; ++a) {
    const int i = cidx[a];
    if (i >= m) {
      const uint64_t u = ctr_rng(seed, RNG_SAMPLE, tcount, ((uint64_t)(uint32_t)s << 32) + (uint64_t)i);
      const int j = (int)(u % (uint64_t)(i + 1));
      if (j < m) atomicMax(&win[j], i);
    }
  }
  __syncthreads();
  for (int j = tid; j < m; j += FWD_THREADS) sel[win[j] >= 0 ? win[j] : j] = 1;
  __syncthreads();
  cnt = 0;
  for (int a = a0; a < a1; ++a) cnt += (cidx[a] < 0 || sel[cidx[a]]) ? 1 : 0;
  int total = 0;
  at = block_excl_scan(cnt, sh_scan, &total);
  for (int a = a0; a < a1; ++a)
    if (cidx[a] < 0 || sel[cidx[a]]) out[at++] = a < ACT_SM ? sh_ids[a] : ids[a];
  __syncthreads();
  for (int a = tid; a < total; a += FWD_THREADS) {
    ids[a] = out[a];
    if (a < ACT_SM) sh_ids[a] = out[a];
  }
  __syncthreads();
  return total;
}

// The sample is skipped: no loss, no gradient, nothing touched (predict: no candidates).
template <int MODE>
__device__ __forceinline__ void skip_sample(const FwdParams& p, int s, int code) {
  const int tid = threadIdx.x;
  if (MODE == 0) {
    for (int k = tid; k < p.H; k += FWD_THREADS) { p.h[(size_t)s * p.H + k] = 0.f; p.dh[(size_t)s * p.H + k] = 0.f; }
    if (tid == 0) { p.act_cnt[s] = 0; p.loss[s] = 0.f; }
  } else {
    for (int q = tid; q < p.topk; q += FWD_THREADS) {
      p.out_ids[(size_t)s * p.topk + q] = -1;
      p.out_scores[(size_t)s * p.topk + q] = -INFINITY;
    }
  }
  if (tid == 0) set_status(p.st, code);
}

// MODE 0 = training step, 1 = predict top-k; KPT = hidden units per thread (H <= KPT * FWD_THREADS); BULK: active sets of
// many chunks are expected (the host's estimate from the tables' shape) and their rows come by bulk copies
template <int MODE, int KPT, bool BULK = false>
__global__ void __launch_bounds__(FWD_THREADS, 2) k_forward(const FwdParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  float* sh_h = reinterpret_cast<float*>(smem);
  float* sh_dh = reinterpret_cast<float*>(smem + p.off_dh);          // [FWD_WARPS][H]
  uint32_t* sh_code = reinterpret_cast<uint32_t*>(smem + p.off_code);
  unsigned char* sh_part = smem + p.off_part;
  int* sh_misc = reinterpret_cast<int*>(smem + p.off_misc);          // 32 ints
  float* sh_red = reinterpret_cast<float*>(sh_misc + 16);
  uint64_t* sh_bar = reinterpret_cast<uint64_t*>(sh_misc + 26);      // 8-byte aligned: off_misc is 16-byte aligned
  uint64_t* sh_bar2 = reinterpret_cast<uint64_t*>(sh_misc + 28);     // completion of the hash functions' mirror
  int* sh_lab = reinterpret_cast<int*>(smem + p.off_lab);            // [max_labels]
  int* sh_tbase = reinterpret_cast<int*>(smem + p.off_tbase);        // [L + 1]
  int* sh_tbeg = reinterpret_cast<int*>(smem + p.off_tbeg);          // [L]
  int* sh_ids = reinterpret_cast<int*>(smem + p.off_ids);            // [ACT_SM]
  float* sh_z = reinterpret_cast<float*>(smem + p.off_z);            // [ACT_SM]
  float* sh_g = reinterpret_cast<float*>(smem + p.off_topk);         // [ACT_SM] training: errors of a small set (predict: its best-k lists)
  int* sh_col = reinterpret_cast<int*>(smem + p.off_col);            // [hid_rows]
  float* sh_val = reinterpret_cast<float*>(smem + p.off_val);        // [hid_rows]
  unsigned char* sh_b1 = smem + p.off_h1;                            // [256] bits of the hidden layer's projections
  int* sh_c1beg = reinterpret_cast<int*>(smem + p.off_h1 + 256);     // [64] start of the slice of every hidden-layer table
  int* sh_c1cnt = sh_c1beg + 64;                                     // [64] and its length
  uint32_t* sh_hmask = reinterpret_cast<uint32_t*>(sh_c1cnt + 64);   // [32] active hidden neurons of the sample
  uint32_t* sh_dd = reinterpret_cast<uint32_t*>(smem + p.off_dedup);
  float* stage = reinterpret_cast<float*>(smem + p.off_dedup);       // overlays the dedup work space

  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, N = p.N;
  // Unless the caller has promised that the batch arrays were complete before the launch, they may still be being
  // written by the kernel before this one in the stream: wait for it before the first read.
  bool waited = false;
  if (!p.inputs_ready) {
    griddep_wait();
    waited = true;
  }
  const int rbeg = p.row_ptr[s], rend = p.row_ptr[s + 1];
  const int nnz = rend - rbeg;
  int lbeg = 0, nlab = 0;
  if (MODE == 0) { lbeg = p.label_ptr[s]; nlab = p.label_ptr[s + 1] - lbeg; }

  griddep_launch_dependents();       // the update kernel may be placed as blocks of this one leave
  if (tid == 0) {
    sh_misc[24] = 0;                 // bucket entries fetched by this sample
    mbar_init(sh_bar, 1);
    mbar_init(sh_bar2, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // the hash functions' tables (constant between rebuilds) come into the upper part of the staging region, which
    // is free until the candidates are collected
    if (p.hash_sm_off >= 0 && !p.dense) {
      mbar_expect_tx(sh_bar2, (uint32_t)p.hash_sm_bytes);
      const int half = p.family == DSLIDE_SIMHASH ? p.hash_sm_bytes / 2 : p.hash_sm_bytes;
      bulk_g2s(smem + p.off_dedup + p.hash_sm_off, p.hash_idx, (uint32_t)half, sh_bar2);
      if (p.family == DSLIDE_SIMHASH) bulk_g2s(smem + p.off_dedup + p.hash_sm_off + half, p.hash_sign, (uint32_t)half, sh_bar2);
    }
  }

  // ---- label checks: ids in range, list within the maximum (merged with the column checks by the first barrier) ----
  int bad = 0;
  if (nnz < 0 || nlab < 0) bad = DSLIDE_ERR_BAD_INDEX;
  else if (MODE == 0) {
    for (int i = tid; i < nlab; i += FWD_THREADS) {
      int y = p.labels[lbeg + i];
      if (y < 0 || y >= N) bad = DSLIDE_ERR_BAD_INDEX;
    }
  }
  const bool too_many_labels = MODE == 0 && nnz >= 0 && nlab > p.max_labels;

  // ---- hidden layer: bias, then one fused multiply-add per nonzero in stored order, ReLU.  The rows of W1 of a
  //      chunk of nonzeros are copied into shared memory together, 16 bytes per thread and copy (cp.async: all of
  //      them in flight at once, no registers held), and then summed per hidden unit in the stored order; the
  //      column ids are checked on the way (in range, ascending) ----
  //      Up to here, and through the first chunk's column ids and values, only the caller's batch is read: with
  //      inputs_ready the kernel runs that far while the previous step's update kernel is still finishing.
  float acc[KPT];
  float s1 = 0.f;                    // sampled hidden layer: the input's sum under projection `tid`
  int c1 = 0, line1 = -1;            // this thread's nonzero (tid-th of the sample), kept for the hand-off to the update kernel
  float x1 = 0.f;
  const int R = p.hid_rows;
  // a thread's place in the copy pattern: 16-byte piece c4 of row r, advancing FWD_THREADS pieces per round
  const int cp_dr = FWD_THREADS / H4, cp_dc = FWD_THREADS - cp_dr * H4;
  const int cp_r0 = tid / H4, cp_c0 = tid - cp_r0 * H4;
  for (int c0 = 0; c0 < nnz; c0 += R) {
    const int nr = min(R, nnz - c0);
    for (int i = tid; i < nr; i += FWD_THREADS) {
      const int c = __ldg(p.col_idx + rbeg + c0 + i);
      const int prev = c0 + i > 0 ? __ldg(p.col_idx + rbeg + c0 + i - 1) : -1;
      const bool okc = c >= 0 && c < p.D && prev < c;
      if (!okc) bad = DSLIDE_ERR_BAD_INDEX;
      sh_col[i] = okc ? c : 0;
      const float xv = __ldg(p.vals + rbeg + c0 + i);
      sh_val[i] = xv;
      if (c0 + i == tid) { c1 = okc ? c : 0; x1 = xv; }
    }
    bad = __syncthreads_or(bad);     // also: the previous chunk's readers of the staging space are done
    if (bad) break;                  // nothing was copied
    if (!waited) {
      griddep_wait();
      waited = true;
    }
    // a feature that has been hot before has a line of the coefficient table (written by the update kernel)
    if (MODE == 0 && c0 == 0 && tid < nr) line1 = __ldcg(p.hotmap1 + c1);
    for (int r = cp_r0, c4 = cp_c0; r < nr;) {
      cp_async16(stage + (size_t)r * H + 4 * c4, p.W1 + (size_t)sh_col[r] * H + 4 * c4);
      c4 += cp_dc; r += cp_dr;
      if (c4 >= H4) { c4 -= H4; ++r; }
    }
    if (c0 == 0) {
#pragma unroll
      for (int u = 0; u < KPT; ++u) {
        const int k = tid + u * FWD_THREADS;
        acc[u] = k < H ? p.b1[k] : 0.f;
      }
    }
    if (p.L1 > 0 && tid < p.KL1) {
      // sampled hidden layer: the input's sum under projection `tid`, nonzeros in stored order (coordinates that the
      // projection does not select add nothing)
      const int8_t* pj = p.proj1 + tid;
      for (int i0 = 0; i0 < nr; i0 += 16) {
        int e[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) e[j] = i0 + j < nr ? (int)__ldg(pj + (size_t)sh_col[i0 + j] * p.KL1) : 0;
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (e[j] != 0) s1 = __fadd_rn(s1, e[j] > 0 ? sh_val[i0 + j] : -sh_val[i0 + j]);
      }
    }
    cp_async_wait_all();
    __syncthreads();
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
      const int k = tid + u * FWD_THREADS;
      if (k < H) {
        float a = acc[u];
#pragma unroll 8
        for (int i = 0; i < nr; ++i) a = __fmaf_rn(sh_val[i], stage[(size_t)i * H + k], a);
        acc[u] = a;
      }
    }
    if (c0 + R < nnz) __syncthreads();       // the next chunk overwrites the column ids and values
  }
  if (nnz <= 0) bad = __syncthreads_or(bad);       // no chunk, no barrier yet: the label checks are merged here
  if (!waited) {                     // no nonzeros, or a bad column id: nothing of the model has been read yet
    griddep_wait();
#pragma unroll
    for (int u = 0; u < KPT; ++u) {
      const int k = tid + u * FWD_THREADS;
      acc[u] = k < H ? p.b1[k] : 0.f;
    }
  }
  if (bad || too_many_labels) {
    if (p.hash_sm_off >= 0 && !p.dense) mbar_wait(sh_bar2, 0u);     // no copy into this block may be left in flight
    skip_sample<MODE>(p, s, (!bad && too_many_labels) ? DSLIDE_ERR_OVERFLOW : DSLIDE_ERR_BAD_INDEX);
    return;
  }
  if (p.L1 > 0) {
    // ---- sampled hidden layer (Algorithm 1: retrieve the layer's active neurons with the layer's input): codes of
    //      the input, one bucket slice per table, union as a bit mask over the hidden neurons.  A neuron that is
    //      not retrieved is a NoOp: activation 0 (Section 2.1) ----
    if (tid < p.KL1) sh_b1[tid] = s1 >= 0.f ? 1 : 0;
    if (tid < 32) sh_hmask[tid] = 0u;
    __syncthreads();
    if (tid < p.L1) {
      uint32_t code = 0;
      for (int k = 0; k < p.K1; ++k) code |= (uint32_t)sh_b1[tid * p.K1 + k] << k;
      if (MODE == 0) p.codes1[(size_t)s * p.L1 + tid] = code;
      const int32_t* off = p.bucket1_off + (size_t)tid * ((1 << p.K1) + 1) + code;
      const int beg = __ldg(off);
      int cnt = __ldg(off + 1) - beg;
      sh_c1beg[tid] = beg;
      sh_c1cnt[tid] = cnt < p.cap1 ? cnt : p.cap1;
    }
    __syncthreads();
    for (int t = warp; t < p.L1; t += FWD_WARPS)
      for (int i = lane; i < sh_c1cnt[t]; i += 32) {
        const int k = __ldg(p.bucket1_ids + (size_t)t * H + sh_c1beg[t] + i);
        atomicOr(&sh_hmask[k >> 5], 1u << (k & 31));
      }
    __syncthreads();
    if (MODE == 0 && tid < p.Hw) p.hmask[(size_t)s * p.Hw + tid] = sh_hmask[tid];
  }
#pragma unroll
  for (int u = 0; u < KPT; ++u) {
    const int k = tid + u * FWD_THREADS;
    if (k < H) {
      const bool on = p.L1 == 0 || ((sh_hmask[k >> 5] >> (k & 31)) & 1u);
      const float hv = (on && acc[u] > 0.f) ? acc[u] : 0.f;
      sh_h[k] = hv;
      if (MODE == 0 || p.dense) p.h[(size_t)s * H + k] = hv;
    }
  }
  if (MODE == 1 && p.dense) return;        // inference over all neurons: the logits are taken by k_predict_dense
  __syncthreads();

  const bool dense = p.dense != 0;
  int na = N;
  int32_t* ids = p.act_ids + (size_t)s * p.act_stride;

  if (!dense) {
    // ---- bucket codes of the hidden activation ----
    const int32_t* hidx = p.hash_idx;
    const int32_t* hsgn = p.hash_sign;
    if (p.hash_sm_off >= 0) {
      const bool ok = mbar_wait(sh_bar2, 0u);
      if (__syncthreads_or(ok ? 0 : 1)) {          // the mirror did not arrive in time: the sample is given up
        mbar_wait(sh_bar2, 0u);
        __syncthreads();
        skip_sample<MODE>(p, s, DSLIDE_ERR_TIMEOUT);
        return;
      }
      hidx = reinterpret_cast<const int32_t*>(smem + p.off_dedup + p.hash_sm_off);
      hsgn = reinterpret_cast<const int32_t*>(smem + p.off_dedup + p.hash_sm_off + p.hash_sm_bytes / 2);
    }
    for (int f = tid; f < p.KL; f += FWD_THREADS) {
      const int32_t* ix = hidx + (size_t)f * p.fn_len;
      if (p.family == DSLIDE_SIMHASH) {
        const int32_t* sg = hsgn + (size_t)f * p.fn_len;
        float sum = 0.f;
        for (int i = 0; i < p.fn_len; ++i) {
          float x = sh_h[ix[i]];
          sum = __fadd_rn(sum, sg[i] > 0 ? x : -x);
        }
        sh_part[f] = sum >= 0.f ? 1 : 0;
      } else if (p.fn_len == 8 && (reinterpret_cast<uintptr_t>(hidx) & 15) == 0) {
        // bins of eight: both halves of the index list in one load each, the eight values fetched side by side
        const int4 ia = reinterpret_cast<const int4*>(ix)[0], ib = reinterpret_cast<const int4*>(ix)[1];
        const float v0 = sh_h[ia.x], v1 = sh_h[ia.y], v2 = sh_h[ia.z], v3 = sh_h[ia.w];
        const float v4 = sh_h[ib.x], v5 = sh_h[ib.y], v6 = sh_h[ib.z], v7 = sh_h[ib.w];
        int best = 0;
        float bv = v0;
        if (v1 > bv) { bv = v1; best = 1; }       // strict: the lowest position wins ties
        if (v2 > bv) { bv = v2; best = 2; }
        if (v3 > bv) { bv = v3; best = 3; }
        if (v4 > bv) { bv = v4; best = 4; }
        if (v5 > bv) { bv = v5; best = 5; }
        if (v6 > bv) { bv = v6; best = 6; }
        if (v7 > bv) { bv = v7; best = 7; }
        sh_part[f] = (unsigned char)best;
        sh_part[p.KL + f] = bv == 0.f ? 1 : 0;     // activations are not negative: a maximum of zero is a bin of zeros
      } else {
        int best = 0;
        float bv = sh_h[ix[0]];
        for (int i = 1; i < p.fn_len; ++i) {
          float v = sh_h[ix[i]];
          if (v > bv) { bv = v; best = i; }       // strict: the lowest position wins ties
        }
        sh_part[f] = (unsigned char)best;
        sh_part[p.KL + f] = bv == 0.f ? 1 : 0;
      }
    }
    __syncthreads();
    // ---- codes, and the slice of every table's bucket the sample reads: all offsets in one round ----
    const int shift = p.family == DSLIDE_SIMHASH ? 1 : p.lg_bin;
    auto table_code = [&](int t) -> uint32_t {
      uint32_t code = 0;
      for (int k = 0; k < p.K; ++k) {
        const int f = t * p.K + k;
        uint32_t pos = sh_part[f];
        if (p.densify && p.family == DSLIDE_DWTA && sh_part[p.KL + f] && p.KL > 1) {
          // a bin of zeros: the position of the first probed function whose own bin is not all zero, else 0
          pos = 0;
          for (int a = 0; a < DENSIFY_ATTEMPTS; ++a) {
            const uint64_t u = ctr_rng(p.seed, RNG_PROBE, p.rcount, (uint64_t)f * DENSIFY_ATTEMPTS + (uint64_t)a);
            const int g = (int)(((uint64_t)f + 1u + u % (uint64_t)(p.KL - 1)) % (uint64_t)p.KL);
            if (!sh_part[p.KL + g]) { pos = sh_part[g]; break; }
          }
        }
        code |= pos << (k * shift);
      }
      return code;
    };
    if (p.L <= 64) {
      // up to 64 tables: one warp fetches all the offsets (two tables per lane) and takes the running sum of the
      // slice lengths in registers -- one barrier instead of two
      if (warp == 0) {
        int beg[2], cnt[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int t = lane + 32 * u;
          beg[u] = 0; cnt[u] = 0;
          if (t < p.L) {
            const uint32_t code = table_code(t);
            sh_code[t] = code;
            if (MODE == 0) p.codes[(size_t)s * p.L + t] = code;
            const int32_t* off = p.bucket_off + (size_t)t * (size_t)(p.nb + 1) + code;
            beg[u] = __ldg(off);
            cnt[u] = __ldg(off + 1);
          }
        }
        int run = 0;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int t = lane + 32 * u;
          int c = cnt[u] - beg[u];
          c = c < p.cap ? c : p.cap;
          int incl = c;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            int n = __shfl_up_sync(FULLM, incl, d);
            if (lane >= d) incl += n;
          }
          if (t < p.L) { sh_tbeg[t] = beg[u]; sh_tbase[t + 1] = run + incl; }
          run += __shfl_sync(FULLM, incl, 31);
        }
        if (lane == 0) { sh_tbase[0] = 0; sh_misc[24] = run; }
      }
      __syncthreads();
    } else {
      for (int t = tid; t < p.L; t += FWD_THREADS) {
        const uint32_t code = table_code(t);
        sh_code[t] = code;
        if (MODE == 0) p.codes[(size_t)s * p.L + t] = code;
        const int32_t* off = p.bucket_off + (size_t)t * (size_t)(p.nb + 1) + code;
        const int beg = __ldg(off);
        int cnt = __ldg(off + 1) - beg;
        cnt = cnt < p.cap ? cnt : p.cap;
        sh_tbeg[t] = beg;
        sh_tbase[t + 1] = cnt;
      }
      __syncthreads();
      if (warp == 0) {            // running sum of the slice lengths: where each table's candidates start
        int run = 0;
        for (int b = 0; b < p.L; b += 32) {
          const int t = b + lane;
          const int v = t < p.L ? sh_tbase[t + 1] : 0;
          int incl = v;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            int n = __shfl_up_sync(FULLM, incl, d);
            if (lane >= d) incl += n;
          }
          if (t < p.L) sh_tbase[t + 1] = run + incl;
          run += __shfl_sync(FULLM, incl, 31);
        }
        if (lane == 0) { sh_tbase[0] = 0; sh_misc[24] = run; }
      }
      __syncthreads();
    }

    // ---- all bucket entries in one round; union over the tables, labels, duplicates removed, ascending ids.
    //      A small candidate set is cheaper to sort than a bitmap over all N neurons is to clear and scan. ----
    const int ncand = sh_tbase[p.L];
    int total = 0;
    const bool bitmap = p.dedup_mode == 1 && ncand + nlab > p.sort_small;
    int n2 = 1;
    if (!bitmap) while (n2 < ncand + nlab) n2 <<= 1;
    // ids short enough to share a word with their position are sorted as such words
    const bool packed = !bitmap && ncand + nlab <= RANK_MAX && N <= (1 << (32 - RANK_BITS));
    if (bitmap) {
      uint4* dd4 = reinterpret_cast<uint4*>(sh_dd);
      const int n4 = (((N + 31) >> 5) + 3) >> 2;
      for (int w = tid; w < n4; w += FWD_THREADS) dd4[w] = make_uint4(0u, 0u, 0u, 0u);
      __syncthreads();
    }
    for (int c = tid; c < ncand; c += FWD_THREADS) {
      int lo = 0, hi = p.L - 1;          // last table whose candidates start at or before c
      while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (sh_tbase[mid] <= c) lo = mid; else hi = mid - 1; }
      const int j = __ldg(p.bucket_ids + (size_t)lo * N + sh_tbeg[lo] + (c - sh_tbase[lo]));
      if (bitmap) atomicOr(&sh_dd[j >> 5], 1u << (j & 31));
      else sh_dd[c] = packed ? ((uint32_t)j << RANK_BITS) | (uint32_t)c : (uint32_t)j;
    }
    if (MODE == 0)
      for (int i = tid; i < nlab; i += FWD_THREADS) {
        const int y = p.labels[lbeg + i];
        if (bitmap) atomicOr(&sh_dd[y >> 5], 1u << (y & 31));
        else sh_dd[ncand + i] = packed ? ((uint32_t)y << RANK_BITS) | (uint32_t)(ncand + i) : (uint32_t)y;
      }
    if (bitmap) {
      __syncthreads();
      const int nwords = (N + 31) >> 5;
      const int chunk = (nwords + FWD_THREADS - 1) / FWD_THREADS;
      const int wbeg = tid * chunk, wend = min(nwords, wbeg + chunk);
      int cnt = 0;
      for (int w = wbeg; w < wend; ++w) cnt += __popc(sh_dd[w]);
      int pos = block_excl_scan(cnt, sh_misc, &total);
      if (total <= p.act_stride && cnt > 0) {
        for (int w = wbeg; w < wend; ++w) {
          uint32_t bits = sh_dd[w];
          while (bits) {
            const int b = __ffs(bits) - 1;
            const int j = (w << 5) + b;
            ids[pos] = j;
            if (pos < ACT_SM) sh_ids[pos] = j;
            ++pos;
            bits &= bits - 1;
          }
        }
      }
    } else if (ncand + nlab <= RANK_MAX) {
      const int n = ncand + nlab;
      if (packed && tid < 4 && n + tid < ((n + 3) & ~3)) sh_dd[n + tid] = 0xffffffffu;
      __syncthreads();
      uint32_t* srt = sh_dd + RANK_MAX;
      const int per = (n + FWD_THREADS - 1) / FWD_THREADS;
      if (packed && n <= FWD_THREADS - 64) {
        // the warps the counting below leaves idle ask L2 for the candidates' rows of W2 meanwhile (the staging after
        // the dedup then finds most of them there); a hint only: duplicates are asked twice, nothing waits for it
        const int idle0 = (n + 31) & ~31;                          // first thread without a value to rank
        const int lines = (H * 4 + 127) >> 7;
        for (int e = tid - idle0; e >= 0 && e < n * (lines + 1); e += FWD_THREADS - idle0) {
          const int c = e / (lines + 1), q = e - c * (lines + 1);
          const int j = (int)(sh_dd[c] >> RANK_BITS);
          prefetch_l2(q < lines ? static_cast<const void*>(p.W2 + (size_t)j * H + 32 * q) : static_cast<const void*>(p.hdr2 + j));
        }
      }
      if (packed) {
        if (per <= 1) rank_sort<1, true>(sh_dd, srt, n);
        else if (per == 2) rank_sort<2, true>(sh_dd, srt, n);
        else rank_sort<RANK_MAX / FWD_THREADS, true>(sh_dd, srt, n);
      } else {
        if (per <= 1) rank_sort<1, false>(sh_dd, srt, n);
        else if (per == 2) rank_sort<2, false>(sh_dd, srt, n);
        else rank_sort<RANK_MAX / FWD_THREADS, false>(sh_dd, srt, n);
      }
      __syncthreads();
      // element i = u * FWD_THREADS + tid of the sorted list is kept when it is the first of its run; its place is
      // the number of kept elements before it: whole rounds and warps (counts exchanged through shared memory) plus
      // the warp's own ballot
      constexpr int PER = RANK_MAX / FWD_THREADS;
      int* sh_cntw = reinterpret_cast<int*>(sh_dh);      // [PER][FWD_WARPS]; the space is not used before the back-propagation
      const unsigned lt = (1u << lane) - 1u;
      const int rounds = (n + FWD_THREADS - 1) / FWD_THREADS;
      unsigned keep[PER];
#pragma unroll
      for (int u = 0; u < PER; ++u) {
        keep[u] = 0u;
        if (u < rounds) {
          const int i = u * FWD_THREADS + tid;
          keep[u] = __ballot_sync(FULLM, i < n && (i == 0 || srt[i - 1] != srt[i]));
          if (lane == 0) sh_cntw[u * FWD_WARPS + warp] = __popc(keep[u]);
        }
      }
      __syncthreads();
      {
        int before = 0;
        for (int q = 0; q < rounds * FWD_WARPS; ++q) {
          const int cq = sh_cntw[q];
          total += cq;
          if (q < warp) before += cq;           // round 0; later rounds add their offset below
        }
        if (total <= p.act_stride) {
          int base = before;
#pragma unroll
          for (int u = 0; u < PER; ++u) {
            if (u < rounds) {
              if (u > 0) {
                base = 0;
                for (int q = 0; q < u * FWD_WARPS + warp; ++q) base += sh_cntw[q];
              }
              const int i = u * FWD_THREADS + tid;
              if ((keep[u] >> lane) & 1u) {
                const int at = base + __popc(keep[u] & lt);
                ids[at] = (int)srt[i];
                if (at < ACT_SM) sh_ids[at] = (int)srt[i];
              }
            }
          }
        }
      }
    } else {
      // sort path: bitonic sort of the candidates, keep the first of each run
      for (int i = ncand + nlab + tid; i < n2; i += FWD_THREADS) sh_dd[i] = 0x7fffffffu;
      __syncthreads();
      for (int k = 2; k <= n2; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
          for (int i = tid; i < n2; i += FWD_THREADS) {
            int x = i ^ j;
            if (x > i) {
              uint32_t a = sh_dd[i], b = sh_dd[x];
              bool asc = (i & k) == 0;
              if ((a > b) == asc) { sh_dd[i] = b; sh_dd[x] = a; }
            }
          }
          __syncthreads();
        }
      const int chunk = (n2 + FWD_THREADS - 1) / FWD_THREADS;
      const int ebeg = tid * chunk, eend = min(n2, ebeg + chunk);
      int cnt = 0;
      for (int i = ebeg; i < eend; ++i) {
        uint32_t a = sh_dd[i];
        cnt += (a != 0x7fffffffu && (i == 0 || sh_dd[i - 1] != a)) ? 1 : 0;
      }
      int pos = block_excl_scan(cnt, sh_misc, &total);
      if (total <= p.act_stride) {
        for (int i = ebeg; i < eend; ++i) {
          uint32_t a = sh_dd[i];
          if (a != 0x7fffffffu && (i == 0 || sh_dd[i - 1] != a)) {
            ids[pos] = (int)a;
            if (pos < ACT_SM) sh_ids[pos] = (int)a;
            ++pos;
          }
        }
      }
    }
    if (total > p.act_stride) {      // uniform over the block
      skip_sample<MODE>(p, s, DSLIDE_ERR_OVERFLOW);
      return;
    }
    na = total;
    __syncthreads();                 // ids visible to the block; the dedup work space is free from here on
    if (p.budget > 0)
      na = budget_select(p.budget, p.budget_fill, N, p.seed, p.tcount, s, ids, sh_ids, na, MODE == 0 ? p.labels + lbeg : nullptr,
                         nlab, smem + p.off_dedup, p.stage_bytes, sh_misc, p.st);
  }
  if (MODE == 0 && tid == 0) p.act_cnt[s] = na;
  const bool small = !dense && na <= ACT_SM;      // ids and logits mirrored in shared memory
  // one pointer per array, to shared or to global memory (a conditional expression over two loads would issue both)
  const int* idp = small ? sh_ids : ids;
  const float* zp = small ? sh_z : p.act_z + (size_t)s * p.act_stride;
  const float* gp = small ? sh_g : p.act_g + (size_t)s * p.act_stride;

  // ---- positions of the sample's distinct labels inside the active set (needed while the rows are staged) ----
  if (MODE == 0) {
    for (int i = tid; i < nlab; i += FWD_THREADS) {
      int y = p.labels[lbeg + i];
      bool first = true;
      for (int q = 0; q < i; ++q) first = first && (p.labels[lbeg + q] != y);
      int pos = y;
      if (!dense) {
        int lo = 0, hi = na;
        while (lo < hi) { int mid = (lo + hi) >> 1; if (idp[mid] < y) lo = mid + 1; else hi = mid; }
        pos = lo;
      }
      sh_lab[i] = first ? pos : -1;
    }
    __syncthreads();
    if (tid == 0) {
      int ny = 0;
      for (int i = 0; i < nlab; ++i) ny += sh_lab[i] >= 0 ? 1 : 0;
      sh_misc[0] = ny;
    }
  }

  // ---- logits over the active set.  The active rows of W2 are copied into shared memory, as many as fit at a
  //      time.  When the whole set fits, the rows stay there for the back-propagation below.  When it does not, the
  //      back-propagated error is accumulated in the same pass, chunk by chunk, with a running maximum M and sums
  //      rescaled whenever M grows: S = sum_a exp(z_a - M) W2[j_a,:], E = sum_a exp(z_a - M), and T = the sum of the
  //      label rows; then dh = (S / E - T / |Y|) / B, and every row is fetched once. ----
  float* z = p.act_z + (size_t)s * p.act_stride;
  float* tk_z = reinterpret_cast<float*>(smem + p.off_topk);          // predict: [FWD_WARPS][topk]
  int* tk_id = reinterpret_cast<int*>(tk_z + FWD_WARPS * p.topk);
  int tk_cnt = 0;                                                     // used by lane 0
  const float4* sh_h4 = reinterpret_cast<const float4*>(sh_h);
  const int ldr = H + 4;                           // staged rows are padded by 16 bytes: a thread per row reads without bank conflicts
  const int stage_rows = p.stage_bytes / (ldr * 4 + 4);      // a row and one float of the chunk's exp(z - M)
  float* sh_ce = stage + (size_t)stage_rows * ldr;           // [stage_rows]
  const bool streaming = MODE == 0 && na > stage_rows;
  float Mrun = -INFINITY, Erun = 0.f;
  float accS[KPT], accT[KPT];
#pragma unroll
  for (int u = 0; u < KPT; ++u) { accS[u] = 0.f; accT[u] = 0.f; }
  const int ngrp = H >= FWD_THREADS ? 1 : min(FWD_WARPS, FWD_THREADS / H);   // groups of H threads (sh_dh holds FWD_WARPS)
  const int grp = H >= FWD_THREADS ? 0 : tid / H;
  // hand-off to the update kernel: the touch counters of the sample's rows of W1 (one per thread) and of its first
  // HO_PER * FWD_THREADS active rows are asked while the first rows of W2 are on their way, the list places after the
  // first logits, and everything is written at the end -- no warp waits for an answer
  constexpr int HO_PER = 2;
  int jj0[HO_PER];
  unsigned nth1 = 0u, nth0[HO_PER], base1 = 0u, base0[HO_PER];
  // a thread's place in the copy pattern of the padded rows: H4 + 1 pieces per row
  const int rp_dr = FWD_THREADS / (H4 + 1), rp_dc = FWD_THREADS - rp_dr * (H4 + 1);
  const int rp_r0 = tid / (H4 + 1), rp_c0 = tid - rp_r0 * (H4 + 1);
#pragma unroll
  for (int u = 0; u < HO_PER; ++u) { jj0[u] = 0; nth0[u] = 0u; base0[u] = 0u; }
  uint32_t w2phase = 0u;
  bool timed_out = false;                          // block-uniform
  const bool bulk = BULK && streaming && na >= 4 * stage_rows;      // many chunks: the batch's samples share most rows (see below)
  for (int c0 = 0; c0 < na; c0 += stage_rows) {
    const int nr = min(stage_rows, na - c0);
    __syncthreads();                               // earlier readers and writers of the staging space are done
    if (bulk) {
      // A set streamed in many chunks re-reads rows that other samples of the batch have brought into L2; there the
      // bulk-copy engine moves about twice what 16-byte copies do per multiprocessor: one copy per row and one for
      // the head of its record (count, bias, bias moments), which lands in the row's padding; completion on an mbarrier
      if (tid == 0) mbar_expect_tx(sh_bar, (uint32_t)nr * ((uint32_t)H * 4u + 16u));
      fence_proxy_async();
      for (int r = tid; r < nr; r += FWD_THREADS) {
        const int j = dense ? c0 + r : idp[c0 + r];
        bulk_g2s(stage + (size_t)r * ldr, p.W2 + (size_t)j * H, (uint32_t)H * 4u, sh_bar);
        bulk_g2s(stage + (size_t)r * ldr + H, p.hdr2 + j, 16u, sh_bar);
      }
    } else {
      // 16 bytes per thread and copy, all in flight at once: the H4 pieces of the row, and as piece H4 the head of
      // the row's record, which lands in the row's padding
      for (int r = rp_r0, c4 = rp_c0; r < nr;) {
        const int j = dense ? c0 + r : idp[c0 + r];
        const void* src = c4 < H4 ? static_cast<const void*>(p.W2 + (size_t)j * H + 4 * c4) : static_cast<const void*>(p.hdr2 + j);
        cp_async16(stage + (size_t)r * ldr + 4 * c4, src);
        c4 += rp_dc; r += rp_dr;
        if (c4 > H4) { c4 -= H4 + 1; ++r; }
      }
    }
    if (c0 == 0 && MODE == 0) {
      // the touch counters: this thread's nonzero of the sample, and its first HO_PER active rows
      if (tid < nnz) {
        if (tid >= R) {                              // beyond the first chunk: not kept in registers above
          c1 = __ldg(p.col_idx + rbeg + tid);
          x1 = __ldg(p.vals + rbeg + tid);
          line1 = __ldcg(p.hotmap1 + c1);
        }
        nth1 = atomicAdd(&p.hdr1[c1].cnt, 1u) & CNT_MASK;
        if (line1 >= 0) p.hotcoef1[(size_t)line1 * p.bstride + s] = x1;
      }
      if (!dense) {
#pragma unroll
        for (int u = 0; u < HO_PER; ++u) {
          const int a = tid + u * FWD_THREADS;
          if (a < na) {
            jj0[u] = idp[a];
            nth0[u] = atomicAdd(&p.hdr2[jj0[u]].cnt, 1u) & CNT_MASK;
          }
        }
      }
    }
    if (bulk) {
      const bool ok = mbar_wait(sh_bar, w2phase);
      w2phase ^= 1u;
      if (__syncthreads_or(ok ? 0 : 1)) { timed_out = true; break; }
    } else {
      cp_async_wait_all();
      __syncthreads();
    }
    // one thread per staged row
    for (int ab = 0; ab < nr; ab += FWD_THREADS) {
      const int a = ab + tid;
      const bool live = a < nr;
      float dot = 0.f;
      if (live) {
        const float4* row = reinterpret_cast<const float4*>(stage + (size_t)a * ldr);
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll 4
        for (int c = 0; c < H4; ++c) {
          const float4 w = row[c], x = sh_h4[c];
          d0 = fmaf(w.x, x.x, d0);
          d1 = fmaf(w.y, x.y, d1);
          d2 = fmaf(w.z, x.z, d2);
          d3 = fmaf(w.w, x.w, d3);
        }
        dot = (d0 + d1) + (d2 + d3);
      }
      if (MODE == 0) {
        if (live) {
          const float zv = stage[(size_t)a * ldr + H + 1] + dot;      // the bias came with the row
          if (small) sh_z[c0 + a] = zv;
          z[c0 + a] = zv;
          if (streaming) sh_ce[a] = zv;
        }
      } else {
        // predict: lane 0 of each warp keeps the warp's best k so far, fed one lane's logit at a time
        int j = -1;
        float zv = 0.f;
        if (live) { j = dense ? c0 + a : idp[c0 + a]; zv = stage[(size_t)a * ldr + H + 1] + dot; }
        float* lz = tk_z + warp * p.topk;
        int* li = tk_id + warp * p.topk;
        // a lane offers its logit only when the list is not full yet or the logit beats the list's last entry
        const int n = __shfl_sync(FULLM, tk_cnt, 0);
        unsigned m = __ballot_sync(FULLM, j >= 0 && (n < p.topk || topk_better(zv, j, lz[p.topk - 1], li[p.topk - 1])));
        while (m) {
          const int l = __ffs(m) - 1;
          m &= m - 1;
          const int jl = __shfl_sync(FULLM, j, l);
          const float zl = __shfl_sync(FULLM, zv, l);
          if (lane == 0 && (tk_cnt < p.topk || topk_better(zl, jl, lz[tk_cnt - 1], li[tk_cnt - 1]))) {
            int q = tk_cnt < p.topk ? tk_cnt++ : p.topk - 1;
            while (q > 0 && topk_better(zl, jl, lz[q - 1], li[q - 1])) { lz[q] = lz[q - 1]; li[q] = li[q - 1]; --q; }
            lz[q] = zl; li[q] = jl;
          }
          __syncwarp();
        }
      }
    }
    if (MODE == 0 && c0 == 0) {
      // the touch counters have answered by now.  W1 side: slot / mask entries (the coefficient is the input value);
      // both sides: places in the lists of distinct rows asked for, used at the end of the kernel
      touch_mark<false>(p, tid < nnz, p.hdr1 + c1, p.mask1 + (size_t)c1 * p.Wd, p.ovf1 + (size_t)c1 * PAIR_T, ~c1, nth1, s, x1);
      base1 = own_reserve(tid < nnz && nth1 == 0u, &p.st->n_own[p.parity][1]);
      if (!dense) {
#pragma unroll
        for (int u = 0; u < HO_PER; ++u)
          if (u * FWD_THREADS < na)          // uniform over the block
            base0[u] = own_reserve(tid + u * FWD_THREADS < na && nth0[u] == 0u, &p.st->n_own[p.parity][0]);
      }
    }
    if (streaming) {
      __syncthreads();
      float cm = -INFINITY;
      for (int a = tid; a < nr; a += FWD_THREADS) cm = fmaxf(cm, sh_ce[a]);
      const float Mnew = fmaxf(Mrun, block_max(cm, sh_red));
      const float scale = expf(Mrun - Mnew);            // 0 for the first chunk
      float es = 0.f;
      for (int a = tid; a < nr; a += FWD_THREADS) {
        const float ea = expf(sh_ce[a] - Mnew);
        sh_ce[a] = ea;
        es += ea;
      }
      Erun = Erun * scale + block_sum(es, sh_red);      // its barriers make the chunk's exp values visible
      Mrun = Mnew;
      if (grp < ngrp) {
#pragma unroll
        for (int u = 0; u < KPT; ++u) {
          const int k = (H >= FWD_THREADS ? tid : tid - grp * H) + u * FWD_THREADS;
          if (k < H && (u == 0 || H > FWD_THREADS)) {
            float v0 = accS[u] * scale, v1 = 0.f, v2 = 0.f, v3 = 0.f;
            int a = grp;
            for (; a + 3 * ngrp < nr; a += 4 * ngrp) {
              v0 = fmaf(sh_ce[a], stage[(size_t)a * ldr + k], v0);
              v1 = fmaf(sh_ce[a + ngrp], stage[(size_t)(a + ngrp) * ldr + k], v1);
              v2 = fmaf(sh_ce[a + 2 * ngrp], stage[(size_t)(a + 2 * ngrp) * ldr + k], v2);
              v3 = fmaf(sh_ce[a + 3 * ngrp], stage[(size_t)(a + 3 * ngrp) * ldr + k], v3);
            }
            for (; a < nr; a += ngrp) v0 = fmaf(sh_ce[a], stage[(size_t)a * ldr + k], v0);
            accS[u] = (v0 + v1) + (v2 + v3);
            if (grp == 0)                               // the label rows of this chunk, once
              for (int i = 0; i < nlab; ++i) {
                const int pos = sh_lab[i] - c0;
                if (sh_lab[i] >= 0 && pos >= 0 && pos < nr) accT[u] += stage[(size_t)pos * ldr + k];
              }
          }
        }
      }
    }
  }
  if (BULK && timed_out) {
    // a copy did not complete in time: the copies in flight get one more bounded wait, then the sample is given up.
    // Its touches are already counted, so the hand-off below still runs, with every coefficient zero.
    mbar_wait(sh_bar, w2phase ^ 1u);
    __syncthreads();
    if (tid == 0) set_status(p.st, DSLIDE_ERR_TIMEOUT);
  }
  if (MODE == 1) {
    // ---- merge the per-warp lists: k rounds over the list heads ----
    if (lane == 0) sh_misc[warp] = tk_cnt;
    __syncthreads();
    if (tid == 0) {
      int head[FWD_WARPS];
      for (int w = 0; w < FWD_WARPS; ++w) head[w] = 0;
      for (int q = 0; q < p.topk; ++q) {
        int bw = -1;
        for (int w = 0; w < FWD_WARPS; ++w) {
          if (head[w] >= sh_misc[w]) continue;
          if (bw < 0 || topk_better(tk_z[w * p.topk + head[w]], tk_id[w * p.topk + head[w]],
                                    tk_z[bw * p.topk + head[bw]], tk_id[bw * p.topk + head[bw]])) bw = w;
        }
        if (bw >= 0) {
          p.out_ids[(size_t)s * p.topk + q] = tk_id[bw * p.topk + head[bw]];
          p.out_scores[(size_t)s * p.topk + q] = tk_z[bw * p.topk + head[bw]];
          head[bw]++;
        } else {
          p.out_ids[(size_t)s * p.topk + q] = -1;
          p.out_scores[(size_t)s * p.topk + q] = -INFINITY;
        }
      }
    }
    return;
  }
  __syncthreads();           // logits visible to the block

  // ---- softmax over the ragged active set, loss, errors.  A small set's logits sit in shared memory: every warp
  //      takes the maximum and the sum over all of them by itself (same order, same result in every warp), which
  //      spares the block-wide reductions and their barriers ----
  float* pr = p.act_p + (size_t)s * p.act_stride;
  float* g = p.act_g + (size_t)s * p.act_stride;
  float M = Mrun, E = Erun;                        // known already when the rows were streamed
  if (!streaming) {
    if (small) {
      float m = -INFINITY;
      for (int a = lane; a < na; a += 32) m = fmaxf(m, sh_z[a]);
      M = warp_max(m);
      float e = 0.f;
      for (int a = lane; a < na; a += 32) e += expf(sh_z[a] - M);
      E = warp_sum(e);
    } else {
      float m = -INFINITY;
      for (int a = tid; a < na; a += FWD_THREADS) m = fmaxf(m, zp[a]);
      M = block_max(m, sh_red);
      float e = 0.f;
      for (int a = tid; a < na; a += FWD_THREADS) e += expf(zp[a] - M);
      E = block_sum(e, sh_red);
    }
  }
  const float fB = (float)p.B;
  const int ny = sh_misc[0];
  if (tid == FWD_THREADS - 1) {                    // the last thread has the fewest rows below
    float sum = 0.f;
    const float logE = logf(E);
    for (int i = 0; i < nlab; ++i)
      if (sh_lab[i] >= 0) sum += zp[sh_lab[i]] - M - logE;
    p.loss[s] = ny > 0 && !(BULK && timed_out) ? -sum / (float)ny : 0.f;
  }
  // the errors of a small set go to shared memory as well (beside the logits: no barrier before they are written)
  for (int a = tid; a < na; a += FWD_THREADS) {
    const float pa = expf(zp[a] - M) / E;
    pr[a] = pa;
    float ga = pa / fB;
    for (int i = 0; i < nlab; ++i)
      if (sh_lab[i] == a) ga = (pa - 1.f / (float)ny) / fB;
    if (BULK && timed_out) ga = 0.f;
    g[a] = ga;
    if (small) sh_g[a] = ga;
  }
  __syncthreads();

  // ---- error at the hidden layer: dh = [h > 0] * sum_a g_a W2[j_a, :] (weights before the update).  Warp w takes
  //      the staged rows w, w + 8, ...; a lane holds four consecutive hidden units of every 128; the warps' sums are
  //      then added in warp order.  When the rows were streamed the sums exist already (per group of threads). ----
  {
    constexpr int NCH = KPT == 1 ? 2 : 2 * MAX_KPT;        // 16-byte pieces of a row per lane: H <= 128 * NCH
    int nparts = ngrp;
    if (!streaming) {
      nparts = FWD_WARPS;
      float4 av[NCH];
#pragma unroll
      for (int q = 0; q < NCH; ++q) av[q] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int a = warp; a < na; a += FWD_WARPS) {
        const float ga = gp[a];
        const float4* row = reinterpret_cast<const float4*>(stage + (size_t)a * ldr);
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
          const int c = lane + 32 * q;
          if (c < H4) {
            const float4 w = row[c];
            av[q].x = fmaf(ga, w.x, av[q].x); av[q].y = fmaf(ga, w.y, av[q].y);
            av[q].z = fmaf(ga, w.z, av[q].z); av[q].w = fmaf(ga, w.w, av[q].w);
          }
        }
      }
#pragma unroll
      for (int q = 0; q < NCH; ++q) {
        const int c = lane + 32 * q;
        if (c < H4) reinterpret_cast<float4*>(sh_dh + (size_t)warp * H)[c] = av[q];
      }
    } else if (grp < ngrp) {
#pragma unroll
      for (int u = 0; u < KPT; ++u) {
        const int k = (H >= FWD_THREADS ? tid : tid - grp * H) + u * FWD_THREADS;
        if (k < H && (u == 0 || H > FWD_THREADS))
          sh_dh[(size_t)grp * H + k] = (accS[u] / E - (ny > 0 ? accT[u] / (float)ny : 0.f)) / fB;
      }
    }
    __syncthreads();
    for (int k = tid; k < H; k += FWD_THREADS) {
      float v = 0.f;
      for (int w = 0; w < nparts; ++w) v += sh_dh[(size_t)w * H + k];
      p.dh[(size_t)s * H + k] = sh_h[k] > 0.f && !(BULK && timed_out) ? v : 0.f;
    }
  }

  // ---- the rest of the hand-off: slot / mask entries of the rows of W2 (their coefficient is the error), the
  //      entries of both lists of distinct rows, and whatever did not fit the registers above ----
  own_store(tid < nnz && nth1 == 0u, base1, p.own1, c1, s);
  if (tid < nnz) list_row(p, &p.hdr1[c1].cnt, ~c1, nth1);
  if (p.L1 > 0)          // sampled hidden layer: of the rows of W1 the sample touches, only its active neurons' weights
    for (int i = tid; i < nnz; i += FWD_THREADS) {
      const int c = i == tid ? c1 : __ldg(p.col_idx + rbeg + i);
      for (int w = 0; w < p.Hw; ++w)
        if (sh_hmask[w]) atomicOr(&p.cmask1[(size_t)c * p.Hw + w], sh_hmask[w]);
    }
  for (int i0 = FWD_THREADS; i0 < nnz; i0 += FWD_THREADS) {
    const int i = i0 + tid;
    const bool live = i < nnz;
    int c = 0;
    unsigned nth = 0u;
    float x = 0.f;
    if (live) {
      c = __ldg(p.col_idx + rbeg + i);
      x = __ldg(p.vals + rbeg + i);
      nth = atomicAdd(&p.hdr1[c].cnt, 1u) & CNT_MASK;
      const int line = __ldg(p.hotmap1 + c);
      if (line >= 0) p.hotcoef1[(size_t)line * p.bstride + s] = x;
    }
    finish_touch(p, live, p.hdr1 + c, p.mask1 + (size_t)c * p.Wd, p.ovf1 + (size_t)c * PAIR_T, p.own1, &p.st->n_own[p.parity][1], c, ~c, nth, s, x);
  }
  if (!dense) {
#pragma unroll
    for (int u = 0; u < HO_PER; ++u)
      if (u * FWD_THREADS < na) {          // uniform over the block
        const int a = tid + u * FWD_THREADS;
        const bool live = a < na;
        touch_mark(p, live, p.hdr2 + jj0[u], p.mask2 + (size_t)jj0[u] * p.Wd, p.ovf2 + (size_t)jj0[u] * PAIR_T, jj0[u], nth0[u], s,
                   live ? gp[a] : 0.f);
        own_store(live && nth0[u] == 0u, base0[u], p.own2, jj0[u], s);
      }
    for (int a0 = HO_PER * FWD_THREADS; a0 < na; a0 += FWD_THREADS) {
      const int a = a0 + tid;
      const bool live = a < na;
      int jj = 0;
      unsigned nth = 0u;
      float ga = 0.f;
      if (live) {
        jj = idp[a];
        ga = gp[a];
        nth = atomicAdd(&p.hdr2[jj].cnt, 1u) & CNT_MASK;
      }
      finish_touch(p, live, p.hdr2 + jj, p.mask2 + (size_t)jj * p.Wd, p.ovf2 + (size_t)jj * PAIR_T, p.own2, &p.st->n_own[p.parity][0], jj, jj, nth, s, ga);
    }
  }
  if (tid == 0) {
    atomicAdd(&p.st->acc[p.parity][0], (unsigned long long)na);
    atomicAdd(&p.st->acc[p.parity][1], (unsigned long long)nnz);
    atomicAdd(&p.st->acc[p.parity][2], (unsigned long long)sh_misc[24]);
  }
}


// ---------------------------------------------------------------------------
// Inference over all N neurons (no tables): logits of PD_SG samples at a time against a slice of W2
// ---------------------------------------------------------------------------
// A block takes PD_SG samples and one slice of the neurons: the samples' hidden activations sit in shared memory, the
// slice's rows pass through the staging space (one bulk copy per row) and every thread takes one staged row against
// all PD_SG activations, so a row is fetched once per PD_SG samples instead of once per sample (PD_SG = 32, 16 or 8,
// the largest whose lists of k fit).  Every warp keeps the
// best k (logit descending, id ascending) per sample in shared memory: a lane offers its logit only when it beats the
// list's last entry.  The block's lists are merged per sample and written out; k_predict_merge merges the slices.
struct PredDenseParams {
  const float* W2;
  const RowHdr* hdr2;
  const float* h;
  DevState* st;
  int32_t* part_ids;     // [nslices][B][k]
  float* part_z;
  int B, H, N, k, nslices, rows_per_round;
};

template <int PD_SG>      // samples per block: more of them means fewer passes over W2, and longer lists in shared memory
__global__ void __launch_bounds__(FWD_THREADS) k_predict_dense(const PredDenseParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, k = p.k, ldr = H + 4;
  float* hs = reinterpret_cast<float*>(smem);                                   // [PD_SG][H]
  float* lz = hs + (size_t)PD_SG * H;                                           // [FWD_WARPS][PD_SG][k]
  int* li = reinterpret_cast<int*>(lz + (size_t)FWD_WARPS * PD_SG * k);
  uint64_t* bar = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(li + (size_t)FWD_WARPS * PD_SG * k) + 15) & ~(uintptr_t)15);
  float* stage = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(bar) + 16);   // [rows_per_round][ldr]
  const int s0 = blockIdx.y * PD_SG;
  const int ns = min(PD_SG, p.B - s0);
  const int per = (p.N + p.nslices - 1) / p.nslices;
  const int jb = min(p.N, (int)blockIdx.x * per), je = min(p.N, jb + per);
  for (int e = tid; e < PD_SG * H; e += FWD_THREADS) {
    const int s = e / H;
    hs[e] = s < ns ? p.h[(size_t)(s0 + s) * H + (e - s * H)] : 0.f;
  }
  if (tid == 0) { mbar_init(bar, 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  int cnt[PD_SG];                          // lane 0: entries in the warp's list of each sample
#pragma unroll
  for (int s = 0; s < PD_SG; ++s) cnt[s] = 0;
  const float4* hs4 = reinterpret_cast<const float4*>(hs);
  uint32_t phase = 0;
  bool timed_out = false;
  for (int r0 = jb; r0 < je; r0 += p.rows_per_round) {
    const int nr = min(p.rows_per_round, je - r0);
    __syncthreads();
    if (tid == 0) mbar_expect_tx(bar, (uint32_t)nr * (uint32_t)H * 4u);
    fence_proxy_async();
    __syncthreads();
    for (int r = tid; r < nr; r += FWD_THREADS)
      bulk_g2s(stage + (size_t)r * ldr, p.W2 + (size_t)(r0 + r) * H, (uint32_t)H * 4u, bar);
    if (!mbar_wait(bar, phase)) timed_out = true;
    phase ^= 1u;
    if (__syncthreads_or(timed_out ? 1 : 0)) { timed_out = true; break; }
    for (int ab = 0; ab < nr; ab += FWD_THREADS) {
      const int a = ab + tid;
      const bool live = a < nr;
      float d[PD_SG];
#pragma unroll
      for (int s = 0; s < PD_SG; ++s) d[s] = 0.f;
      float bias = 0.f;
      if (live) {
        bias = __ldg(&p.hdr2[r0 + a].b);
        const float4* row = reinterpret_cast<const float4*>(stage + (size_t)a * ldr);
        for (int c = 0; c < H4; ++c) {
          const float4 w = row[c];
#pragma unroll
          for (int s = 0; s < PD_SG; ++s) {
            const float4 x = hs4[s * H4 + c];
            d[s] = fmaf(w.x, x.x, d[s]); d[s] = fmaf(w.y, x.y, d[s]); d[s] = fmaf(w.z, x.z, d[s]); d[s] = fmaf(w.w, x.w, d[s]);
          }
        }
      }
      const int j = r0 + a;
#pragma unroll
      for (int s = 0; s < PD_SG; ++s) {
        if (s >= ns) break;                                   // uniform
        const float z = bias + d[s];
        float* wz = lz + ((size_t)warp * PD_SG + s) * k;
        int* wi = li + ((size_t)warp * PD_SG + s) * k;
        const int n = __shfl_sync(FULLM, cnt[s], 0);
        const bool offer = live && (n < k || topk_better(z, j, wz[k - 1], wi[k - 1]));
        unsigned m = __ballot_sync(FULLM, offer);
        while (m) {                                           // rare once the lists have filled
          const int l = __ffs(m) - 1;
          m &= m - 1;
          const float zl = __shfl_sync(FULLM, z, l);
          const int jl = __shfl_sync(FULLM, j, l);
          if (lane == 0 && (cnt[s] < k || topk_better(zl, jl, wz[cnt[s] - 1], wi[cnt[s] - 1]))) {
            int q = cnt[s] < k ? cnt[s]++ : k - 1;
            while (q > 0 && topk_better(zl, jl, wz[q - 1], wi[q - 1])) { wz[q] = wz[q - 1]; wi[q] = wi[q - 1]; --q; }
            wz[q] = zl; wi[q] = jl;
          }
          __syncwarp();
        }
      }
    }
  }
  if (timed_out) {
    mbar_wait(bar, phase ^ 1u);
    if (tid == 0) set_status(p.st, DSLIDE_ERR_TIMEOUT);
  }
  // the eight warps' lists of a sample, merged by one thread per sample: k rounds over the list heads
  int* sh_cnt = reinterpret_cast<int*>(stage);                // [FWD_WARPS][PD_SG] (the staging space is free now)
  __syncthreads();
  if (lane == 0)
#pragma unroll
    for (int s = 0; s < PD_SG; ++s) sh_cnt[warp * PD_SG + s] = timed_out ? 0 : cnt[s];
  __syncthreads();
  if (tid < ns) {
    const int s = tid;
    int head[FWD_WARPS];
    for (int w = 0; w < FWD_WARPS; ++w) head[w] = 0;
    int32_t* oi = p.part_ids + ((size_t)blockIdx.x * p.B + (s0 + s)) * k;
    float* oz = p.part_z + ((size_t)blockIdx.x * p.B + (s0 + s)) * k;
    for (int q = 0; q < k; ++q) {
      int bw = -1;
      for (int w = 0; w < FWD_WARPS; ++w) {
        if (head[w] >= sh_cnt[w * PD_SG + s]) continue;
        const float* wz = lz + ((size_t)w * PD_SG + s) * k;
        const int* wi = li + ((size_t)w * PD_SG + s) * k;
        if (bw < 0) { bw = w; continue; }
        const float* bz = lz + ((size_t)bw * PD_SG + s) * k;
        const int* bi = li + ((size_t)bw * PD_SG + s) * k;
        if (topk_better(wz[head[w]], wi[head[w]], bz[head[bw]], bi[head[bw]])) bw = w;
      }
      if (bw >= 0) {
        oi[q] = li[((size_t)bw * PD_SG + s) * k + head[bw]];
        oz[q] = lz[((size_t)bw * PD_SG + s) * k + head[bw]];
        head[bw]++;
      } else {
        oi[q] = -1;
        oz[q] = -INFINITY;
      }
    }
  }
}

// One thread per sample merges the slices' lists (each in order, padded with id -1).
__global__ void k_predict_merge(const int32_t* part_ids, const float* part_z, int B, int k, int nslices, int32_t* out_ids,
                                float* out_scores) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= B) return;
  int head[64];
  for (int w = 0; w < nslices; ++w) head[w] = 0;
  for (int q = 0; q < k; ++q) {
    int bw = -1;
    for (int w = 0; w < nslices; ++w) {
      if (head[w] >= k) continue;
      const size_t at = ((size_t)w * B + s) * k + head[w];
      if (part_ids[at] < 0) continue;
      if (bw < 0) { bw = w; continue; }
      const size_t bt = ((size_t)bw * B + s) * k + head[bw];
      if (topk_better(part_z[at], part_ids[at], part_z[bt], part_ids[bt])) bw = w;
    }
    if (bw >= 0) {
      const size_t bt = ((size_t)bw * B + s) * k + head[bw];
      out_ids[(size_t)s * k + q] = part_ids[bt];
      out_scores[(size_t)s * k + q] = part_z[bt];
      head[bw]++;
    } else {
      out_ids[(size_t)s * k + q] = -1;
      out_scores[(size_t)s * k + q] = -INFINITY;
    }
  }
}

// ---------------------------------------------------------------------------
// Host side: shared-memory layout and launches
// ---------------------------------------------------------------------------
static int align16(int x) { return (x + 15) & ~15; }
static int align128(int x) { return (x + 127) & ~127; }

struct FwdLayout {
  int off_dh, off_code, off_part, off_misc, off_lab, off_tbase, off_tbeg, off_topk, off_ids, off_z, off_col, off_val,
      off_h1, off_dedup, fixed_bytes, hid_rows;
};

static FwdLayout fwd_layout(const Ctx* c) {
  FwdLayout l;
  // rows of W1 staged per chunk of the hidden layer: HID_MIN_BYTES worth, between 8 and 128
  int hid_rows = HID_MIN_BYTES / (c->H * 4);
  if (hid_rows > 128) hid_rows = 128;
  if (hid_rows < 8) hid_rows = 8;
  l.hid_rows = hid_rows;
  int o = align16(c->H * 4);
  l.off_dh = o;      o = align16(o + FWD_WARPS * c->H * 4);
  l.off_code = o;    o = align16(o + c->L * 4);
  l.off_part = o;    o = align16(o + 2 * c->KL);     // position and all-zero flag of every function's bin
  l.off_misc = o;    o = align16(o + 32 * 4);
  l.off_lab = o;     o = align16(o + (c->cfg.max_labels > 0 ? c->cfg.max_labels : 1) * 4);
  l.off_tbase = o;   o = align16(o + (c->L + 1) * 4);
  l.off_tbeg = o;    o = align16(o + c->L * 4);
  l.off_topk = o;    o = align16(o + FWD_WARPS * 64 * 8);
  l.off_ids = o;     o = align16(o + ACT_SM * 4);
  l.off_z = o;       o = align16(o + ACT_SM * 4);
  l.off_col = o;     o = align16(o + hid_rows * 4);
  l.off_val = o;     o = align16(o + hid_rows * 4);
  l.off_h1 = o;      o = align16(o + 256 + 64 * 4 * 2 + 32 * 4);     // sampled hidden layer: bits, slice starts and lengths, active mask
  o = align128(o);
  l.off_dedup = o;
  l.fixed_bytes = o;
  return l;
}

cudaError_t setup_forward(Ctx* c) {
  FwdLayout l = fwd_layout(c);
  const int budget = 227 * 1024 - l.fixed_bytes;
  const int bitmap_bytes = align16(((c->N + 31) / 32) * 4);
  int64_t worst = (int64_t)c->L * c->cap + c->cfg.max_labels;
  int64_t pow2 = 1;
  while (pow2 < worst) pow2 <<= 1;
  const int64_t sort_bytes = pow2 * 4;
  // the staging space holds the hidden layer's chunk of W1 rows and, later, active rows of W2
  const int stage_min = l.hid_rows * c->H * 4;
  int mode = c->cfg.dedup_mode;
  int dd_bytes = 0;
  if (c->dense) { mode = 1; c->sort_cap = 0; }
  else {
    if (mode == 0) mode = (bitmap_bytes <= 100 * 1024 || sort_bytes > budget) ? 1 : 2;
    if (mode == 1 && bitmap_bytes > budget) return cudaErrorInvalidValue;
    if (mode == 2 && sort_bytes > budget) return cudaErrorInvalidValue;
    c->sort_cap = (int)pow2;
    dd_bytes = mode == 1 ? bitmap_bytes : (int)sort_bytes;
  }
  c->dedup_mode = mode;
  int stage = dd_bytes > stage_min ? dd_bytes : stage_min;
  // when the dedup work space leaves room for two blocks per multiprocessor, staging gets the rest of a half
  const int two_per_sm = (227 * 1024) / 2 - 1024 - l.fixed_bytes;
  if (stage < two_per_sm) stage = two_per_sm;
  if (stage > budget) stage = budget;
  if (stage < stage_min || stage < c->H * 4) return cudaErrorInvalidValue;
  c->fwd_stage_bytes = stage & ~15;
  // dedup by sorting for small candidate sets: mode 0 picks per sample, mode 1 always uses the bitmap, mode 2 always sorts
  c->fwd_sort_small = 0;
  if (mode == 1 && c->cfg.dedup_mode == 0 && !c->dense) {
    int cap_small = c->fwd_stage_bytes / 8;      // the sort pads to a power of two
    c->fwd_sort_small = cap_small < SORT_SMALL ? cap_small : SORT_SMALL;
  }
  // the hash functions' tables are mirrored above the hidden layer's chunk when they fit there
  {
    const long long one = (long long)c->KL * c->fn_len * 4;
    const long long hb = c->cfg.hash_family == DSLIDE_SIMHASH ? 2 * one : one;
    c->fwd_hash_sm_off = -1;
    c->fwd_hash_sm_bytes = 0;
    if (!c->dense && one % 16 == 0 && hb <= 32 * 1024 && stage_min + hb <= (long long)c->fwd_stage_bytes) {
      c->fwd_hash_sm_bytes = (int)hb;
      c->fwd_hash_sm_off = (c->fwd_stage_bytes - (int)hb) & ~15;
    }
  }
  if (c->cfg.sample_budget > 0 && !c->dense) {
    // the reservoir's work space (an index per retrieved id, a slot per kept one, flags, the kept ids) overlays the staging region
    const long long a = c->act_stride, m = c->cfg.sample_budget < c->act_stride ? c->cfg.sample_budget : c->act_stride;
    if (4 * a + 4 * m + a + 16 + 4 * (m + c->cfg.max_labels) > (long long)c->fwd_stage_bytes) return cudaErrorInvalidValue;
    if (c->cfg.budget_fill) {
      // the fill's work space for the largest number of missing ids (the whole budget): draws, flags, hash set, ids
      const long long b = c->cfg.sample_budget < c->N ? c->cfg.sample_budget : c->N, D = 2 * b + 64;
      long long ts = 64;
      while (ts < 2 * D) ts <<= 1;
      if (4 * D + D + 4 + 8 * ts + 8 * b + 4 * b > (long long)c->fwd_stage_bytes) return cudaErrorInvalidValue;
    }
  }
  c->fwd_smem = l.fixed_bytes + c->fwd_stage_bytes;
  cudaError_t e = cudaFuncSetAttribute(k_forward<0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_forward<0, MAX_KPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_forward<0, 1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_forward<0, MAX_KPT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_forward<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_forward<1, MAX_KPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  return e;
}

static FwdParams make_params(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                             const int32_t* label_ptr, const int32_t* labels) {
  FwdParams p;
  p.W1 = c->W1; p.b1 = c->b1; p.W2 = c->W2;
  p.hash_idx = c->hash_idx; p.hash_sign = c->hash_sign; p.bucket_off = c->bucket_off; p.bucket_ids = c->bucket_ids;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.vals = vals; p.label_ptr = label_ptr; p.labels = labels;
  p.h = c->h; p.dh = c->dh; p.loss = c->loss; p.codes = c->codes;
  p.act_cnt = c->act_cnt; p.act_ids = c->act_ids; p.act_z = c->act_z; p.act_p = c->act_p; p.act_g = c->act_g;
  p.mask1 = c->mask1; p.mask2 = c->mask2; p.ovf1 = c->ovf1; p.ovf2 = c->ovf2;
  p.hotmap1 = c->hotmap1; p.hotcoef1 = c->hotcoef1; p.bstride = c->cfg.max_batch; p.hdr1 = c->hdr1; p.hdr2 = c->hdr2;
  p.own1 = c->own1; p.own2 = c->own2; p.hot_rows = c->hot_rows; p.med_rows = c->med_rows; p.parity = (int)(c->t_host & 1);
  p.st = c->dstate; p.out_ids = nullptr; p.out_scores = nullptr;
  p.nb = c->nb;
  p.B = batch; p.D = c->D; p.H = c->H; p.N = c->N; p.K = c->K; p.L = c->L; p.KL = c->KL;
  p.family = c->cfg.hash_family; p.lg_bin = c->lg_bin; p.fn_len = c->fn_len; p.cap = c->cap;
  p.act_stride = c->act_stride; p.Wd = c->Wd; p.dense = c->dense; p.dedup_mode = c->dedup_mode;
  p.max_labels = c->cfg.max_labels; p.sort_cap = c->sort_cap; p.topk = 1;
  FwdLayout l = fwd_layout(c);
  p.stage_bytes = c->fwd_stage_bytes; p.hid_rows = l.hid_rows; p.sort_small = c->fwd_sort_small;
  p.densify = c->cfg.dwta_densify; p.seed = c->cfg.seed; p.rcount = (unsigned long long)c->r_host;
  p.budget = c->cfg.sample_budget; p.budget_fill = c->cfg.budget_fill; p.tcount = (unsigned long long)c->t_host;
  p.hash_sm_off = c->fwd_hash_sm_off; p.hash_sm_bytes = c->fwd_hash_sm_bytes; p.inputs_ready = 1;
  p.off_dh = l.off_dh; p.off_code = l.off_code; p.off_part = l.off_part; p.off_misc = l.off_misc;
  p.off_lab = l.off_lab; p.off_tbase = l.off_tbase; p.off_tbeg = l.off_tbeg; p.off_topk = l.off_topk;
  p.off_ids = l.off_ids; p.off_z = l.off_z; p.off_col = l.off_col; p.off_val = l.off_val; p.off_dedup = l.off_dedup;
  p.off_h1 = l.off_h1;
  p.proj1 = c->proj1; p.bucket1_off = c->bucket1_off; p.bucket1_ids = c->bucket1_ids;
  p.codes1 = c->codes1; p.hmask = c->hmask; p.cmask1 = c->cmask1;
  p.K1 = c->K1; p.L1 = c->L1; p.KL1 = c->KL1; p.cap1 = c->cap1; p.Hw = c->Hw;
  return p;
}

cudaError_t launch_forward_train(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                                 const int32_t* label_ptr, const int32_t* labels, int inputs_ready) {
  FwdParams p = make_params(c, batch, row_ptr, col_idx, vals, label_ptr, labels);
  p.inputs_ready = inputs_ready;
  {
    LaunchScope ls(c, KID_FORWARD);
    // hidden layers of up to FWD_THREADS units take the variant with one unit per thread (less code, fewer registers)
    // Expected size of an active set from the tables' shape: L buckets of about N / 2^bits ids, cut at the cap (and at
    // the sampling budget).  Sets of many chunks of the staging space take the variant that fetches rows by bulk copies.
    const double per_bucket = (double)c->N / (double)(1ll << c->bits);
    double expect = c->cfg.force_dense ? (double)c->N : (double)c->L * (per_bucket < c->cfg.bucket_cap ? per_bucket : (double)c->cfg.bucket_cap);
    if (c->cfg.sample_budget > 0 && expect > c->cfg.sample_budget) expect = c->cfg.sample_budget;
    const bool bulk = expect >= 4.0 * (double)(p.stage_bytes / ((c->H + 4) * 4 + 4));
    cudaError_t e;
    if (c->H <= FWD_THREADS)
      e = bulk ? launch_dependent(k_forward<0, 1, true>, dim3(batch), dim3(FWD_THREADS), (size_t)c->fwd_smem, c->stream, p)
               : launch_dependent(k_forward<0, 1>, dim3(batch), dim3(FWD_THREADS), (size_t)c->fwd_smem, c->stream, p);
    else
      e = bulk ? launch_dependent(k_forward<0, MAX_KPT, true>, dim3(batch), dim3(FWD_THREADS), (size_t)c->fwd_smem, c->stream, p)
               : launch_dependent(k_forward<0, MAX_KPT>, dim3(batch), dim3(FWD_THREADS), (size_t)c->fwd_smem, c->stream, p);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t launch_predict(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                           int k, int dense, int32_t* out_ids, float* out_scores) {
  FwdParams p = make_params(c, batch, row_ptr, col_idx, vals, nullptr, nullptr);
  p.topk = k;
  p.out_ids = out_ids;
  p.out_scores = out_scores;
  if (dense) p.dense = 1;
  LaunchScope ls(c, KID_PREDICT);
  if (c->H <= FWD_THREADS) k_forward<1, 1><<<batch, FWD_THREADS, c->fwd_smem, c->stream>>>(p);
  else k_forward<1, MAX_KPT><<<batch, FWD_THREADS, c->fwd_smem, c->stream>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || !dense) return e;
  // over all neurons: the kernel above has left the hidden activations.  Small k on supported shapes: the tensor pipe
  // filters the candidates and an exact pass orders them; otherwise groups of sg samples x slices of W2 on the ALUs
  if (dense_tc_usable(c, k)) return launch_dense_tc(c, batch, k, out_ids, out_scores);
  const int sg = k <= 8 ? 32 : (k <= 16 ? 16 : 8);
  const int ngroups = (batch + sg - 1) / sg;
  int nslices = (2 * c->num_sms + ngroups - 1) / ngroups;
  if (nslices > 64) nslices = 64;
  if (nslices > c->N) nslices = c->N;
  if (nslices < 1) nslices = 1;
  const size_t need = (size_t)nslices * batch * k * 8;
  if (need > c->pd_cap) {
    if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) return e;
    if (c->pd_part) cudaFree(c->pd_part);
    c->pd_part = nullptr; c->pd_cap = 0;
    if ((e = cudaMalloc(&c->pd_part, need)) != cudaSuccess) return e;
    c->pd_cap = need;
  }
  PredDenseParams q;
  q.W2 = c->W2; q.hdr2 = c->hdr2; q.h = c->h; q.st = c->dstate;
  q.part_ids = reinterpret_cast<int32_t*>(c->pd_part);
  q.part_z = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(c->pd_part) + (size_t)nslices * batch * k * 4);
  q.B = batch; q.H = c->H; q.N = c->N; q.k = k; q.nslices = nslices;
  const size_t fixed = (size_t)sg * c->H * 4 + (size_t)FWD_WARPS * sg * k * 8 + 48;
  const size_t row = (size_t)(c->H + 4) * 4;
  long long rows = ((long long)(227 * 1024) / 2 - (long long)fixed - 1024) / (long long)row;     // two blocks per multiprocessor
  if (rows < 8) rows = ((long long)(227 * 1024) - (long long)fixed - 1024) / (long long)row;
  if (rows < 1) return cudaErrorInvalidValue;
  if (rows > 512) rows = 512;
  q.rows_per_round = (int)rows;
  const size_t smem = fixed + (size_t)rows * row;
  auto kern = sg == 32 ? k_predict_dense<32> : (sg == 16 ? k_predict_dense<16> : k_predict_dense<8>);
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)) != cudaSuccess) return e;
  kern<<<dim3(nslices, ngroups), FWD_THREADS, smem, c->stream>>>(q);
  k_predict_merge<<<(batch + 127) / 128, 128, 0, c->stream>>>(q.part_ids, q.part_z, batch, k, nslices, out_ids, out_scores);
  return cudaGetLastError();
}

}  // namespace dslide
