// Update kernels of the SLIDE step (Algorithm 1 "Update weights with Adam"; Section 3.5: a
// momentum and a velocity array per weight and bias array; Section 2.1: gradients reach the
// active neurons only).
//
// The forward kernel leaves, per step and per touched row of W2 / W1: in the row's 64-byte record the
// number of samples that touch the row and the (sample, coefficient) pairs of its first ROW_SLOTS
// touches (the record also holds the bias of a row of W2 with its moments, so one line brings all of
// it); a bit mask of the samples of any further touches, whose pairs up to touch PAIR_T are kept in a
// side array as well; and two lists of (row, first-touching sample) for the distinct touched rows.
//
//   k_update : a warp works on two rows of the row lists at a time; the loads of a row's weights and
//              moments, of its record and of the first-touching sample's row (h for W2, dh for W1) are
//              all issued together.  A row touched by one sample takes its gradient from slot 0; a row
//              touched by up to ROW_SLOTS samples from its slots, put in ascending sample order; a row
//              touched by up to PAIR_T samples from its slots and kept pairs, likewise; a row touched by
//              more from slots and mask (the sample's coefficient for this row is found by binary
//              search in the sample's ascending id list), again in ascending sample order.  So
//              the sums do not depend on the order in which the forward kernel's blocks ran, and no
//              floating-point atomics are used.  Rows touched by more than ROW_SLOTS samples were
//              listed by the forward kernel and are summed by a warp each; rows touched by more than
//              HOT_T samples were listed a second time: each is cut into HOT_SLICES slices of its mask,
//              summed by different warps, and the warp that finishes a row's last slice adds the slice
//              sums in slice order (rows of W1 that have been hot before find their coefficients in a
//              table line the forward kernel fills, instead of searching).  Warps draw tickets (the first two are fixed by the warp's number,
//              the others come from a counter): hot slices, then listed rows, then the ordinary rows four
//              at a time, the last few thousand two at a time.  Adam is applied to the touched rows only; untouched rows are neither read
//              nor written.  The warp that updates a row resets its count and mask for the next step.
//              The first blocks of the grid update the hidden bias and reduce the batch loss.
//   k_adam_dense : the output layer when every neuron is active (no lists, no masks).
#include "common.cuh"

namespace dslide {

constexpr int UPD_THREADS = 256;
constexpr int UPD_WARPS = UPD_THREADS / 32;
constexpr unsigned FULL = 0xffffffffu;
// ROW_SLOTS (common.cuh): touches of a row whose (sample, coefficient) the forward kernel stores directly

struct UpdParams {
  float *W1, *mW1, *vW1, *b1, *mb1, *vb1;
  float *W2, *mW2, *vW2;
  const float *h, *dh, *act_g, *loss;
  const int32_t *act_cnt, *act_ids;
  const int32_t *row_ptr, *col_idx;
  const float* vals;
  uint32_t *mask1, *mask2;
  const int2 *ovf1, *ovf2;
  int32_t* hotmap1;
  const float* hotcoef1;
  int bstride;
  RowHdr *hdr1, *hdr2;
  const int2 *own1, *own2;
  const int32_t *hot_rows, *med_rows;
  float* hot_part;
  int* hot_done;
  DevState* st;
  float* loss_out;
  HostResult* host_res;        // mapped host memory that receives {status, loss, sequence number}, or null
  unsigned int host_seq;
  int B, H, N, D, Wd, act_stride, dense, parity;
  float lr, beta1, beta2, eps, rb1, rb2;
  // LSH-sampled hidden layer (L1 > 0): per row of W1 the hidden units some sample touches it for; per sample its active units
  uint32_t* cmask1;
  const uint32_t* hmask;
  int L1, Hw;
};

// One element of Adam.  rb1 = 1 / (1 - beta1^t), rb2 = 1 / (1 - beta2^t).  The square root and the final
// quotient use the hardware approximations (relative error below 2^-22): three orders of magnitude inside
// the fp32 noise of the gradient sums, and free of the slow paths exact zeros take in the IEEE sequences.
__device__ __forceinline__ void adam1(float& w, float& m, float& v, float g, float b1, float b2, float lr, float eps,
                                      float rb1, float rb2) {
  m = fmaf(b1, m, (1.f - b1) * g);
  v = fmaf(b2, v, (1.f - b2) * g * g);
  float root;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(v * rb2));
  w = w - __fdividef(lr * (m * rb1), root + eps);
}

__device__ __forceinline__ void axpy4(float4& a, float g, const float4 x) {
  a.x = fmaf(g, x.x, a.x); a.y = fmaf(g, x.y, a.y); a.z = fmaf(g, x.z, a.z); a.w = fmaf(g, x.w, a.w);
}

// The pieces of one layer's update: the weight / moment arrays, the rows that multiply the
// coefficients (h for W2, dh for W1), the per-row masks and the per-row records (touch count, slots and,
// for W2, the bias with its moments).
// Asks L2 for `bytes` (a multiple of 16, from a 16-byte boundary); nothing comes back to the multiprocessor.
__device__ __forceinline__ void l2_fetch(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

struct Side {
  float *W, *M, *V;
  const float* src;
  uint32_t* mask;
  const int2* ovf;
  RowHdr* hdr;
  int is_w2;
};

__device__ __forceinline__ Side make_side(const UpdParams& p, bool w2) {
  Side sd;
  sd.W = w2 ? p.W2 : p.W1; sd.M = w2 ? p.mW2 : p.mW1; sd.V = w2 ? p.vW2 : p.vW1;
  sd.src = w2 ? p.h : p.dh;
  sd.mask = w2 ? p.mask2 : p.mask1;
  sd.ovf = w2 ? p.ovf2 : p.ovf1;
  sd.hdr = w2 ? p.hdr2 : p.hdr1;
  sd.is_w2 = w2 ? 1 : 0;
  return sd;
}

// Coefficient of (row, sample s): the error of neuron `row` in sample s, or the value of feature
// `row` in sample s.  Both lists are ascending, so a binary search finds it.
__device__ __forceinline__ float find_coef(const UpdParams& p, const Side& sd, const int* rowptr, int row, int s) {
  if (sd.is_w2) {
    const int32_t* ids = p.act_ids + (size_t)s * p.act_stride;
    const int n = p.act_cnt[s];
    int lo = 0, hi = n;
    while (lo < hi) { int mid = (lo + hi) >> 1; if (__ldg(ids + mid) < row) lo = mid + 1; else hi = mid; }
    return (lo < n && __ldg(ids + lo) == row) ? __ldg(p.act_g + (size_t)s * p.act_stride + lo) : 0.f;
  }
  int lo = __ldg(rowptr + s);
  const int end = __ldg(rowptr + s + 1);
  int hi = end;
  while (lo < hi) { int mid = (lo + hi) >> 1; if (__ldg(p.col_idx + mid) < row) lo = mid + 1; else hi = mid; }
  return (lo < end && __ldg(p.col_idx + lo) == row) ? __ldg(p.vals + lo) : 0.f;
}

// acc += sum over the set bits b of `bits` (ascending) of coef[b] * src[(sbase + b) * H ...], where coef[b]
// lives in lane b.  Up to four rows are loaded before they are used, in order.
template <int NCH>
__device__ __forceinline__ void accumulate_word(float4 (&acc)[NCH], float& csum, uint32_t bits, float coef,
                                                int sbase, const float* src, int H, int H4, int lane) {
  while (bits) {
    int b[4]; float g[4]; int n = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      b[r] = -1; g[r] = 0.f;
      if (bits) { b[r] = __ffs(bits) - 1; bits &= bits - 1; n = r + 1; }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) g[r] = __shfl_sync(FULL, coef, b[r] < 0 ? 0 : b[r]);
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
      int c = lane + q * 32;
      if (c < H4) {
        float4 x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
          x[r] = r < n ? __ldg(reinterpret_cast<const float4*>(src + (size_t)(sbase + b[r]) * H) + c)
                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 0; r < 4; ++r) if (r < n) axpy4(acc[q], g[r], x[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) if (r < n) csum += g[r];
  }
}

// acc += sum_{k < n} coef_k * src[s_k * H ...] in the order k = 0, 1, ..., where lane k holds (s_k, coef_k).
// Up to four rows are loaded before they are used, in order.
template <int NCH>
__device__ __forceinline__ void accumulate_list(float4 (&acc)[NCH], float& csum, int n, int s_mine, float g_mine,
                                                const float* src, int H, int H4, int lane) {
  for (int k0 = 0; k0 < n; k0 += 4) {
    int sr[4]; float g[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int k = k0 + r < n ? k0 + r : 0;
      sr[r] = __shfl_sync(FULL, s_mine, k);
      g[r] = __shfl_sync(FULL, g_mine, k);
    }
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
      int c = lane + q * 32;
      if (c < H4) {
        float4 x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
          x[r] = k0 + r < n ? __ldg(reinterpret_cast<const float4*>(src + (size_t)sr[r] * H) + c)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 0; r < 4; ++r) if (k0 + r < n) axpy4(acc[q], g[r], x[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) if (k0 + r < n) csum += g[r];
  }
}

// Gradient of a row touched by 2..ROW_SLOTS samples: the (sample, coefficient) pairs of its slots, put in
// ascending sample order through the warp's scratch.
template <int NCH>
__device__ __forceinline__ void sum_slots(const Side& sd, int2 sl, int total, int* scr, float4 (&acc)[NCH],
                                          float& csum, int H, int H4, int lane) {
  if (lane >= total) sl.x = 0x7fffffff;
  int rank = 0;
#pragma unroll
  for (int k = 0; k < ROW_SLOTS; ++k) {
    const int sk = __shfl_sync(FULL, sl.x, k);
    rank += (k < total && sk < sl.x) ? 1 : 0;
  }
  __syncwarp();
  if (lane < total) { scr[rank] = sl.x; scr[32 + rank] = sl.y; }
  __syncwarp();
  const int s_mine = lane < total ? scr[lane] : 0;
  const float g_mine = lane < total ? __int_as_float(scr[32 + lane]) : 0.f;
  accumulate_list<NCH>(acc, csum, total, s_mine, g_mine, sd.src, H, H4, lane);
}

// Gradient of a row touched by more than ROW_SLOTS samples, restricted to the samples of the mask words
// [w0, w1): the samples of the slots and of the mask, ascending.  Up to 32 samples at a time are listed
// in the warp's scratch, their coefficients looked up in parallel, then added in order.  Clears the mask.
template <int NCH>
__device__ __forceinline__ void sum_masked(const UpdParams& p, const Side& sd, const int* rowptr, int row,
                                           int slot_s, int w0, int w1, int* scr, float4 (&acc)[NCH], float& csum,
                                           int H, int H4, int lane, const float* line = nullptr) {
  uint32_t* mrow = sd.mask + (size_t)row * p.Wd;
  int fill = 0;
  const unsigned lt = (1u << lane) - 1u;
  for (int wb = w0; wb < w1; wb += 32) {
    const int wi = wb + lane;
    uint32_t word = wi < w1 ? mrow[wi] : 0u;
    if (word) mrow[wi] = 0u;                     // clean for the next step
#pragma unroll
    for (int k = 0; k < ROW_SLOTS; ++k) {
      const int sk = __shfl_sync(FULL, slot_s, k);
      if (wi < w1 && (sk >> 5) == wi) word |= 1u << (sk & 31);
    }
    unsigned nz = __ballot_sync(FULL, word != 0u);
    while (nz) {
      const int srcl = __ffs(nz) - 1;
      nz &= nz - 1;
      const uint32_t bits = __shfl_sync(FULL, word, srcl);
      const int nb = __popc(bits);
      if (fill + nb > 32) {
        __syncwarp();
        const int s_mine = lane < fill ? scr[lane] : 0;
        const float g_mine = lane < fill ? (line ? line[s_mine] : find_coef(p, sd, rowptr, row, s_mine)) : 0.f;
        accumulate_list<NCH>(acc, csum, fill, s_mine, g_mine, sd.src, H, H4, lane);
        fill = 0;
        __syncwarp();
      }
      if ((bits >> lane) & 1u) scr[fill + __popc(bits & lt)] = ((wb + srcl) << 5) + lane;
      fill += nb;
    }
  }
  __syncwarp();
  if (fill > 0) {
    const int s_mine = lane < fill ? scr[lane] : 0;
    const float g_mine = lane < fill ? (line ? line[s_mine] : find_coef(p, sd, rowptr, row, s_mine)) : 0.f;
    accumulate_list<NCH>(acc, csum, fill, s_mine, g_mine, sd.src, H, H4, lane);
  }
  __syncwarp();
}

template <int NCH>
__device__ __forceinline__ void load_row(const float* base, size_t row, int H, int H4, int lane, float4 (&x)[NCH]) {
  const float4* r4 = reinterpret_cast<const float4*>(base + row * H);
#pragma unroll
  for (int q = 0; q < NCH; ++q) {
    int c = lane + q * 32;
    x[q] = c < H4 ? r4[c] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

template <int NCH, bool UMASK = false>      // UMASK: rows of W1 carry a mask of the hidden units to update (sampled hidden layer)
__device__ __forceinline__ void adam_store(const UpdParams& p, const Side& sd, size_t row, float4 (&w)[NCH],
                                           float4 (&m)[NCH], float4 (&v)[NCH], const float4 (&g)[NCH], int H, int H4,
                                           int lane) {
  float4* w4 = reinterpret_cast<float4*>(sd.W + row * H);
  float4* m4 = reinterpret_cast<float4*>(sd.M + row * H);
  float4* v4 = reinterpret_cast<float4*>(sd.V + row * H);
  // a row of W1 under a sampled hidden layer: only the units some sample touched the row for are updated (the
  // others keep weight and moments bit for bit); the row's unit mask is cleared by finish_hdr
  const uint32_t* um = (UMASK && !sd.is_w2) ? p.cmask1 + row * (size_t)p.Hw : nullptr;
#pragma unroll
  for (int q = 0; q < NCH; ++q) {
    int c = lane + q * 32;
    if (c < H4) {
      if (UMASK) {
        unsigned on = 0xfu;
        if (um) on = (um[(4 * c) >> 5] >> ((4 * c) & 31)) & 0xfu;
        if (on & 1u) adam1(w[q].x, m[q].x, v[q].x, g[q].x, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        if (on & 2u) adam1(w[q].y, m[q].y, v[q].y, g[q].y, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        if (on & 4u) adam1(w[q].z, m[q].z, v[q].z, g[q].z, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        if (on & 8u) adam1(w[q].w, m[q].w, v[q].w, g[q].w, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
      } else {
        adam1(w[q].x, m[q].x, v[q].x, g[q].x, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        adam1(w[q].y, m[q].y, v[q].y, g[q].y, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        adam1(w[q].z, m[q].z, v[q].z, g[q].z, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
        adam1(w[q].w, m[q].w, v[q].w, g[q].w, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
      }
      w4[c] = w[q];
      __stcs(m4 + c, m[q]);      // the moments are not read again before the next update of this row
      __stcs(v4 + c, v[q]);
    }
  }
}

// A row record as a warp holds it: lane l < 8 has the l-th 8-byte piece -- lane 0 (count, bias), lane 1 (the
// bias moments), lanes 2.. the slots.
__device__ __forceinline__ int2 load_hdr(const RowHdr* hd, int lane) {
  int2 v = make_int2(0, 0);
  if (lane < 8) v = reinterpret_cast<const int2*>(hd)[lane];
  return v;
}
// Slot k of the record in lane k (k < ROW_SLOTS).
__device__ __forceinline__ int2 hdr_slots(int2 hv) {
  return make_int2(__shfl_down_sync(FULL, hv.x, 2), __shfl_down_sync(FULL, hv.y, 2));
}
// Closes a row: Adam on the bias of a row of W2 with the gradient g, and the touch count back to zero for the
// next step.  Called by the whole warp.
__device__ __forceinline__ void finish_hdr(const UpdParams& p, RowHdr* hd, bool w2, int2 hv, float g, int lane) {
  if (w2) {
    float b = __int_as_float(__shfl_sync(FULL, hv.y, 0));
    float mb = __int_as_float(__shfl_sync(FULL, hv.x, 1));
    float vb = __int_as_float(__shfl_sync(FULL, hv.y, 1));
    adam1(b, mb, vb, g, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
    if (lane == 0) reinterpret_cast<int2*>(hd)[0] = make_int2(0, __float_as_int(b));
    if (lane == 1) reinterpret_cast<int2*>(hd)[1] = make_int2(__float_as_int(mb), __float_as_int(vb));
  } else {
    if (lane == 0) hd->cnt = 0u;
    if (p.L1 > 0 && lane < p.Hw) p.cmask1[(size_t)(hd - p.hdr1) * p.Hw + lane] = 0u;     // the row's unit mask, for the next step
  }
}

// The hidden bias (dense gradient, summed over the samples in eight fixed slices) and, in the first
// of these blocks, the mean loss and the step statistics.
__device__ void aux_block(const UpdParams& p, int a, float* sm_part, unsigned* sm_on) {     // sm_on: UPD_WARPS * 32 words
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, B = p.B;
  const int k = a * 32 + lane;
  const int per = (B + UPD_WARPS - 1) / UPD_WARPS;
  const int s0 = warp * per, s1 = min(B, s0 + per);
  float g = 0.f;
  unsigned any_on = p.L1 > 0 ? 0u : 1u;        // sampled hidden layer: was unit k active for any sample?
  if (k < H && p.L1 > 0)
    for (int s = s0; s < s1; ++s) any_on |= (p.hmask[(size_t)s * p.Hw + (k >> 5)] >> (k & 31)) & 1u;
  if (k < H) {
    int s = s0;
    for (; s + 8 <= s1; s += 8) {
      float x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = p.dh[(size_t)(s + u) * H + k];
#pragma unroll
      for (int u = 0; u < 8; ++u) g += x[u];
    }
    for (; s < s1; ++s) g += p.dh[(size_t)s * H + k];
  }
  sm_part[warp * 32 + lane] = g;
  sm_on[warp * 32 + lane] = any_on;
  __syncthreads();
  if (warp == 0 && k < H) {
    float tot = 0.f;
    unsigned on = 0u;
    for (int w = 0; w < UPD_WARPS; ++w) { tot += sm_part[w * 32 + lane]; on |= sm_on[w * 32 + lane]; }
    if (on) {
      float w = p.b1[k], m = p.mb1[k], v = p.vb1[k];
      adam1(w, m, v, tot, p.beta1, p.beta2, p.lr, p.eps, p.rb1, p.rb2);
      p.b1[k] = w; p.mb1[k] = m; p.vb1[k] = v;
    }
  }
  if (a != 0) return;
  __syncthreads();
  // mean loss of the batch, summed in a fixed order
  float v = 0.f;
  for (int s = tid; s < B; s += UPD_THREADS) v += p.loss[s];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(FULL, v, d);
  if (lane == 0) sm_part[warp] = v;
  __syncthreads();
  if (tid == 0) {
    float r = 0.f;
    for (int w = 0; w < UPD_WARPS; ++w) r += sm_part[w];
    if (p.loss_out) *p.loss_out = r / (float)B;
    DevState* st = p.st;
    if (p.host_res) {            // the forward kernel has finished: the sticky status covers this step
      p.host_res->status = st->status;
      p.host_res->loss = r / (float)B;
      __threadfence_system();
      *reinterpret_cast<volatile unsigned int*>(&p.host_res->seq) = p.host_seq;
    }
    const int q = p.parity, o = q ^ 1;
    st->last[0] = st->acc[q][0]; st->last[1] = st->acc[q][1]; st->last[2] = st->acc[q][2];
    st->cum[0] += 1ull; st->cum[1] += st->acc[q][0]; st->cum[4] += st->acc[q][1]; st->cum[5] += st->acc[q][2];
    if (p.dense) st->cum[2] += (unsigned long long)p.N;
    // the other parity's slots are the next step's: start them at zero
    st->acc[o][0] = 0ull; st->acc[o][1] = 0ull; st->acc[o][2] = 0ull;
    st->cum[3] += (unsigned long long)st->n_own[q][1];
    if (!p.dense) st->cum[2] += (unsigned long long)st->n_own[q][0];
    st->n_own[o][0] = 0u; st->n_own[o][1] = 0u; st->n_hot[o] = 0u; st->n_med[o] = 0u; st->ticket[o] = 0u;
  }
}

// One slice of a row touched by many samples: the samples of HOT_SLICES-th of the row's mask words.  The slice
// sum goes to scratch memory; the warp that completes the row's last slice adds the slices in slice
// order (so the result does not depend on which warp that is), applies Adam and resets the row's state.
template <int NCH, bool UMASK>
__device__ __forceinline__ void hot_item(const UpdParams& p, const int* rowptr, int item, int nwB, int* scr, int H,
                                         int H4, int lane) {
  const int hrow = item / HOT_SLICES, slice = item - hrow * HOT_SLICES;
  const int code = p.hot_rows[hrow];
  const bool w2 = code >= 0;
  const int row = w2 ? code : ~code;
  const Side sd = make_side(p, w2);
  const int per_w = (nwB + HOT_SLICES - 1) / HOT_SLICES;
  const int w0 = min(nwB, slice * per_w), w1 = min(nwB, w0 + per_w);
  float4 acc[NCH];
#pragma unroll
  for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  float csum = 0.f;
  const int2 hv = load_hdr(sd.hdr + row, lane);
  // a row of W1 that has been hot before has its coefficients in its line of the table (left there by the forward
  // kernel of this step), indexed by sample: no search
  const int hline = w2 ? -1 : p.hotmap1[row];
  sum_masked<NCH>(p, sd, rowptr, row, hdr_slots(hv).x, w0, w1, scr, acc, csum, H, H4, lane,
                  hline >= 0 ? p.hotcoef1 + (size_t)hline * p.bstride : nullptr);
  const int ld = H + 4;
  float* part = p.hot_part + (size_t)hrow * HOT_SLICES * ld;
  float4* mine = reinterpret_cast<float4*>(part + (size_t)slice * ld);
#pragma unroll
  for (int u = 0; u < NCH; ++u) {
    const int c = lane + u * 32;
    if (c < H4) __stcg(mine + c, acc[u]);
  }
  if (lane == 0) __stcg(part + (size_t)slice * ld + H, csum);
  __threadfence();
  __syncwarp();
  int done = 0;
  if (lane == 0) done = atomicAdd(p.hot_done + hrow, 1);
  done = __shfl_sync(FULL, done, 0);
  if (done != HOT_SLICES - 1) return;
  __threadfence();
  float4 w[NCH], m[NCH], v[NCH];
  load_row<NCH>(sd.W, (size_t)row, H, H4, lane, w);
  load_row<NCH>(sd.M, (size_t)row, H, H4, lane, m);
  load_row<NCH>(sd.V, (size_t)row, H, H4, lane, v);
#pragma unroll
  for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  csum = 0.f;
  for (int sl = 0; sl < HOT_SLICES; ++sl) {
    const float4* src4 = reinterpret_cast<const float4*>(part + (size_t)sl * ld);
#pragma unroll
    for (int u = 0; u < NCH; ++u) {
      const int c = lane + u * 32;
      if (c < H4) {
        const float4 x = __ldcg(src4 + c);
        acc[u].x += x.x; acc[u].y += x.y; acc[u].z += x.z; acc[u].w += x.w;
      }
    }
    csum += __ldcg(part + (size_t)sl * ld + H);
  }
  adam_store<NCH, UMASK>(p, sd, (size_t)row, w, m, v, acc, H, H4, lane);
  finish_hdr(p, sd.hdr + row, w2, hv, csum, lane);
  if (lane == 0) {
    p.hot_done[hrow] = 0;
    if (!w2 && hline < 0) {           // hot for the first time: a line for the steps to come (every slice of this step has read -1)
      const unsigned at = atomicAdd(&p.st->n_hotslots, 1u);
      if (at < (unsigned)HOTMAP_CAP) p.hotmap1[row] = (int)at;
    }
  }
}

// A row touched by more than ROW_SLOTS samples that the forward kernel listed: one warp sums it from slots and
// mask (ascending samples), applies Adam and resets the row's state.  Rows that went on to the hot list are
// summed in slices instead and skipped here.
template <int NCH, bool UMASK>
__device__ __forceinline__ void medium_item(const UpdParams& p, const int* rowptr, int idx, int nwB, int* scr, int H,
                                            int H4, int lane) {
  const int code = p.med_rows[idx];
  const bool w2 = code >= 0;
  const int row = w2 ? code : ~code;
  const Side sd = make_side(p, w2);
  const int2 hv = load_hdr(sd.hdr + row, lane);
  const unsigned cv = (unsigned)__shfl_sync(FULL, hv.x, 0);
  if ((cv & CNT_HOT) || (cv & CNT_MASK) == 0u) return;
  const int2 sl = hdr_slots(hv);
  const int total = (int)(cv & CNT_MASK);
  // the pairs of touches ROW_SLOTS .. PAIR_T - 1, asked for together with the rows
  int2 pair = sl;
  if (total <= PAIR_T && lane >= ROW_SLOTS && lane < total) pair = sd.ovf[(size_t)row * PAIR_T + lane];
  float4 w[NCH], m[NCH], v[NCH], acc[NCH];
  load_row<NCH>(sd.W, (size_t)row, H, H4, lane, w);
  load_row<NCH>(sd.M, (size_t)row, H, H4, lane, m);
  load_row<NCH>(sd.V, (size_t)row, H, H4, lane, v);
#pragma unroll
  for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  float csum = 0.f;
  if (total <= PAIR_T) {
    // every touch has its pair: lane k holds touch k; put them in ascending sample order (each sample touches a
    // row once, so the samples are distinct) and add; the mask only has to be cleared
    const int s_me = lane < total ? pair.x : 0x7fffffff;
    int rank = 0;
    for (int k = 0; k < total; ++k) rank += __shfl_sync(FULL, s_me, k) < s_me ? 1 : 0;
    __syncwarp();
    if (lane < total) { scr[rank] = pair.x; scr[32 + rank] = pair.y; }
    __syncwarp();
    const int s_mine = lane < total ? scr[lane] : 0;
    const float g_mine = lane < total ? __int_as_float(scr[32 + lane]) : 0.f;
    accumulate_list<NCH>(acc, csum, total, s_mine, g_mine, sd.src, H, H4, lane);
    __syncwarp();
    uint32_t* mrow = sd.mask + (size_t)row * p.Wd;
    for (int wi = lane; wi < nwB; wi += 32)
      if (mrow[wi]) mrow[wi] = 0u;
  } else {
    sum_masked<NCH>(p, sd, rowptr, row, sl.x, 0, nwB, scr, acc, csum, H, H4, lane);
  }
  adam_store<NCH, UMASK>(p, sd, (size_t)row, w, m, v, acc, H, H4, lane);
  finish_hdr(p, sd.hdr + row, w2, hv, csum, lane);
}

// Work is handed out in tickets from one counter: first the slices of the hot rows (the longest items), then
// the listed rows with more than ROW_SLOTS touches, then the ordinary rows, UPD_TROWS per ticket (small tickets keep the tail of the kernel short).
constexpr int UPD_TROWS = 4;

template <int NCH, int G, bool UMASK>
__global__ void __launch_bounds__(UPD_THREADS, (NCH == 1 ? 2 : (NCH == 2 ? 2 : 1))) k_update(const UpdParams p) {
  extern __shared__ __align__(16) unsigned char upd_smem[];
  const int* rowptr = p.row_ptr;      // the batch's row offsets (read through the read-only path where needed)
  float* sm_part = reinterpret_cast<float*>(upd_smem);   // [UPD_WARPS * 32]
  __shared__ int scratch[UPD_WARPS][64];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, B = p.B;
  const int naux = (H + 31) >> 5;
  // the next step's forward kernel may be placed as blocks of this one leave; everything this kernel reads was
  // written by the forward kernel before it
  griddep_launch_dependents();
  griddep_wait();
  if ((int)blockIdx.x < naux) { aux_block(p, (int)blockIdx.x, sm_part, reinterpret_cast<unsigned*>(&scratch[0][0])); return; }


  const int n2 = p.dense ? 0 : (int)p.st->n_own[p.parity][0];
  const int n1 = (int)p.st->n_own[p.parity][1];
  const int nrows = n2 + n1;
  const int nwB = (B + 31) >> 5;
  const unsigned nh_raw = p.st->n_hot[p.parity], nm_raw = p.st->n_med[p.parity];
  const int n_hot_items = (int)(nh_raw < (unsigned)HOT_CAP ? nh_raw : (unsigned)HOT_CAP) * HOT_SLICES;
  const int n_med = (int)(nm_raw < (unsigned)MED_CAP ? nm_raw : (unsigned)MED_CAP);
  // ordinary rows go out UPD_TROWS per ticket, except the last few thousand, which go out G per ticket so that the
  // warps finish close together
  const int nwork = (int)gridDim.x - naux;
  const int nwarps = nwork * UPD_WARPS;
  const int rows_small = min(nrows, UPD_TROWS * nwarps);
  const int rows_big = (nrows - rows_small) / UPD_TROWS * UPD_TROWS;
  const int n_big = rows_big / UPD_TROWS;
  const int n_norm = n_big + (nrows - rows_big + G - 1) / G;
  const int n_tickets = n_hot_items + n_med + n_norm;
  unsigned int* ticket = &p.st->ticket[p.parity];

  // a warp's first two tickets are fixed by its number; further tickets come from the counter, each asked for a
  // whole ticket before it is needed
  int cur = warp * nwork + ((int)blockIdx.x - naux);
  int nxt = nwarps + cur;
  int fut = 0;
  if (lane == 0) fut = 2 * nwarps + (int)atomicAdd(ticket, 1u);
  // The list entries of a warp's next ticket are read while it works on the current one, and the rows they name are
  // asked into L2 (a ticket's time ahead of their use: the loads of the next ticket then wait for L2, not for DRAM).
  int2 nrow = make_int2(0, 0);
  int nidx = nrows, nfor = -1;         // the entries held are those of ticket nfor
  auto entries_of = [&](int t, int2& row, int& idx) {
    row = make_int2(0, 0);
    idx = nrows;
    const int k = t - n_hot_items - n_med;
    if (t >= n_tickets || k < 0) return;
    const int first = k < n_big ? k * UPD_TROWS : rows_big + (k - n_big) * G;
    const int trows = k < n_big ? UPD_TROWS : G;
    if (lane < trows && first + lane < nrows) {
      idx = first + lane;
      row = idx < n2 ? p.own2[idx] : p.own1[idx - n2];
    }
  };
  for (;; cur = nxt, nxt = __shfl_sync(FULL, fut, 0), fut = (lane == 0 && nxt < n_tickets) ? 2 * nwarps + (int)atomicAdd(ticket, 1u) : fut) {
    const int t = cur;
    if (t >= n_tickets) break;
    if (t < n_hot_items) { hot_item<NCH, UMASK>(p, rowptr, t, nwB, scratch[warp], H, H4, lane); continue; }
    if (t < n_hot_items + n_med) { medium_item<NCH, UMASK>(p, rowptr, t - n_hot_items, nwB, scratch[warp], H, H4, lane); continue; }

    // ---- ordinary rows: consecutive entries of the concatenated lists (rows of W2, then rows of W1) ----
    const int trows = t - n_hot_items - n_med < n_big ? UPD_TROWS : G;
    int2 myrow = nrow;                   // (row, the sample that touched it first = the sample of slot 0)
    int myidx = nidx;
    if (NCH > 1 || nfor != t) entries_of(t, myrow, myidx);
    if (NCH == 1) {                      // rows of up to 512 bytes; with longer rows the kernel is near the copy bandwidth
      entries_of(nxt, nrow, nidx);       // and looking ahead only adds load.  Used after this ticket's own loads are issued
      nfor = nxt;
    }
    for (int b0 = 0; b0 < trows; b0 += G) {
      int rr[G], tt[G];
      bool live[G], w2[G], skip[G];
      int2 hv[G], sl[G];
      float4 w[G][NCH], m[G][NCH], v[G][NCH], x[G][NCH];
#pragma unroll
      for (int q = 0; q < G; ++q) {
        const int idx = __shfl_sync(FULL, myidx, b0 + q);
        live[q] = idx < nrows;
        w2[q] = idx < n2;
        rr[q] = __shfl_sync(FULL, myrow.x, b0 + q);
        const int s0 = __shfl_sync(FULL, myrow.y, b0 + q);
        tt[q] = 0;
        hv[q] = make_int2(0, 0);
        if (live[q]) {
          const Side sd = make_side(p, w2[q]);
          hv[q] = load_hdr(sd.hdr + rr[q], lane);
          load_row<NCH>(sd.src, (size_t)s0, H, H4, lane, x[q]);      // the row of slot 0's sample: all a once-touched row needs
          load_row<NCH>(sd.W, (size_t)rr[q], H, H4, lane, w[q]);
          load_row<NCH>(sd.M, (size_t)rr[q], H, H4, lane, m[q]);
          load_row<NCH>(sd.V, (size_t)rr[q], H, H4, lane, v[q]);
        }
      }
      if (NCH == 1 && b0 == 0 && nidx < nrows) {
        const Side sn = make_side(p, nidx < n2);
        const uint32_t bytes = (uint32_t)H * 4u;
        l2_fetch(sn.W + (size_t)nrow.x * H, bytes);
        l2_fetch(sn.M + (size_t)nrow.x * H, bytes);
        l2_fetch(sn.V + (size_t)nrow.x * H, bytes);
        l2_fetch(sn.hdr + nrow.x, (uint32_t)sizeof(RowHdr));
      }
#pragma unroll
      for (int q = 0; q < G; ++q)
        if (live[q]) {
          const unsigned cv = (unsigned)__shfl_sync(FULL, hv[q].x, 0);
          sl[q] = hdr_slots(hv[q]);
          // a listed row is summed by its own ticket (and its count may already be back at zero)
          skip[q] = (cv & (CNT_HOT | CNT_MED)) != 0u || (cv & CNT_MASK) == 0u;
          tt[q] = (int)(cv & CNT_MASK);
        }
#pragma unroll
      for (int q = 0; q < G; ++q)
        if (live[q] && !skip[q]) {
          const Side sd = make_side(p, w2[q]);
          float4 acc[NCH];
#pragma unroll
          for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          float csum = 0.f;
          if (tt[q] == 1) {
            const float g0 = __int_as_float(__shfl_sync(FULL, sl[q].y, 0));
#pragma unroll
            for (int u = 0; u < NCH; ++u) axpy4(acc[u], g0, x[q][u]);
            csum = g0;
          } else if (tt[q] <= ROW_SLOTS) {
            sum_slots<NCH>(sd, sl[q], tt[q], scratch[warp], acc, csum, H, H4, lane);
          } else {      // more touches than slots, yet not listed (the list was full)
            sum_masked<NCH>(p, sd, rowptr, rr[q], sl[q].x, 0, nwB, scratch[warp], acc, csum, H, H4, lane);
          }
          adam_store<NCH, UMASK>(p, sd, (size_t)rr[q], w[q], m[q], v[q], acc, H, H4, lane);
          finish_hdr(p, sd.hdr + rr[q], w2[q], hv[q], csum, lane);
        }
    }
  }
}

// Output layer with every neuron active: one warp per row of W2, samples summed in ascending order.
constexpr int DENSE_CH = 8;
__global__ void __launch_bounds__(UPD_THREADS) k_adam_dense(const UpdParams p) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, B = p.B;
  const Side sd = make_side(p, true);
  for (int j = blockIdx.x * UPD_WARPS + warp; j < p.N; j += gridDim.x * UPD_WARPS) {
    float4 acc[DENSE_CH];
#pragma unroll
    for (int q = 0; q < DENSE_CH; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    float csum = 0.f;
    for (int sb = 0; sb < B; sb += 32) {
      const int s = sb + lane;
      // a skipped sample has an empty active set and contributes nothing
      const float coef = (s < B && p.act_cnt[s] > 0) ? p.act_g[(size_t)s * p.act_stride + j] : 0.f;
      const uint32_t bits = B - sb >= 32 ? 0xffffffffu : ((1u << (B - sb)) - 1u);
      accumulate_word<DENSE_CH>(acc, csum, bits, coef, sb, p.h, H, H4, lane);
    }
    float4 w[DENSE_CH], m[DENSE_CH], v[DENSE_CH];
    load_row<DENSE_CH>(sd.W, (size_t)j, H, H4, lane, w);
    load_row<DENSE_CH>(sd.M, (size_t)j, H, H4, lane, m);
    load_row<DENSE_CH>(sd.V, (size_t)j, H, H4, lane, v);
    adam_store<DENSE_CH>(p, sd, (size_t)j, w, m, v, acc, H, H4, lane);
    finish_hdr(p, sd.hdr + j, true, load_hdr(sd.hdr + j, lane), csum, lane);
  }
}

template <int NCH, int G, bool UMASK>
static cudaError_t launch_k_update(Ctx* c, const UpdParams& p, int smem) {
  cudaError_t e = cudaSuccess;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(k_update<NCH, G, UMASK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  // the kernel needs little shared memory: the rest of the unified store serves as cache for the h / dh rows
  e = cudaFuncSetAttribute(k_update<NCH, G, UMASK>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxL1);
  if (e != cudaSuccess) return e;
  // one wave: the blocks for the hidden bias come first, the rest fill the remaining block slots of the device
  const int naux = (c->H + 31) / 32;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_update<NCH, G, UMASK>, UPD_THREADS, smem);
  if (e != cudaSuccess) return e;
  int nblocks = c->num_sms * (per_sm > 0 ? per_sm : 1);
  if (nblocks < naux + 1) nblocks = naux + 1;
  LaunchScope ls(c, KID_ADAM);
  e = launch_dependent(k_update<NCH, G, UMASK>, dim3(nblocks), dim3(UPD_THREADS), (size_t)smem, c->stream, p);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

cudaError_t launch_update(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                          float* loss_out, HostResult* host_res, unsigned int host_seq) {
  UpdParams p;
  p.W1 = c->W1; p.mW1 = c->mW1; p.vW1 = c->vW1; p.b1 = c->b1; p.mb1 = c->mb1; p.vb1 = c->vb1;
  p.W2 = c->W2; p.mW2 = c->mW2; p.vW2 = c->vW2;
  p.h = c->h; p.dh = c->dh; p.act_g = c->act_g; p.loss = c->loss; p.act_cnt = c->act_cnt; p.act_ids = c->act_ids;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.vals = vals;
  p.mask1 = c->mask1; p.mask2 = c->mask2; p.ovf1 = c->ovf1; p.ovf2 = c->ovf2;
  p.hotmap1 = c->hotmap1; p.hotcoef1 = c->hotcoef1; p.bstride = c->cfg.max_batch; p.hdr1 = c->hdr1; p.hdr2 = c->hdr2;
  p.own1 = c->own1; p.own2 = c->own2;
  p.hot_rows = c->hot_rows; p.med_rows = c->med_rows; p.hot_part = c->hot_part; p.hot_done = c->hot_done;
  p.st = c->dstate; p.loss_out = loss_out; p.host_res = host_res; p.host_seq = host_seq;
  p.B = batch; p.H = c->H; p.N = c->N; p.D = c->D; p.Wd = c->Wd; p.act_stride = c->act_stride; p.dense = c->dense;
  p.parity = (int)(c->t_host & 1);
  p.cmask1 = c->cmask1; p.hmask = c->hmask; p.L1 = c->L1; p.Hw = c->Hw;
  p.lr = c->cfg.lr; p.beta1 = c->cfg.beta1; p.beta2 = c->cfg.beta2; p.eps = c->cfg.eps;
  // reciprocal bias corrections of Adam with the global step count (the step being taken is t + 1)
  const double t = (double)(c->t_host + 1);
  p.rb1 = (float)(1.0 / (1.0 - pow((double)c->cfg.beta1, t)));
  p.rb2 = (float)(1.0 / (1.0 - pow((double)c->cfg.beta2, t)));

  if (c->dense) {
    LaunchScope ls(c, KID_ADAM_DENSE);
    k_adam_dense<<<c->num_sms * 4, UPD_THREADS, 0, c->stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int smem = UPD_WARPS * 32 * 4;
  const int nch = (c->H / 4 + 31) / 32;
  if (c->L1 > 0) {        // sampled hidden layer: rows of W1 are updated under their unit masks
    if (nch <= 1) return launch_k_update<1, 2, true>(c, p, smem);
    if (nch <= 2) return launch_k_update<2, 2, true>(c, p, smem);
    if (nch <= 4) return launch_k_update<4, 1, true>(c, p, smem);
    return launch_k_update<8, 1, true>(c, p, smem);
  }
  if (nch <= 1) return launch_k_update<1, 2, false>(c, p, smem);
  if (nch <= 2) return launch_k_update<2, 2, false>(c, p, smem);
  if (nch <= 4) return launch_k_update<4, 1, false>(c, p, smem);
  return launch_k_update<8, 1, false>(c, p, smem);
}

}  // namespace dslide
