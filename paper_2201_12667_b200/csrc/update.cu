// Update kernels of the SLIDE step (Algorithm 1 "Update weights with Adam"; Section 3.5: a
// momentum and a velocity array per weight and bias array; Section 2.1: gradients reach the
// active neurons only).
//
// The forward kernel leaves, per step and per touched row of W2 / W1: the number of samples that
// touch the row, the (sample, coefficient) pairs of its first ROW_SLOTS touches, a bit mask of the
// samples of any further touches -- and two lists of the distinct touched rows (the sample that
// touched a row first entered it).
//
//   k_update : every warp takes a contiguous share of the two row lists, a few rows at a time, so
//              that the loads of a row's weights and moments, its touch count and its slots are
//              all issued together.  A row touched by one sample takes its gradient from slot 0;
//              a row touched by up to ROW_SLOTS samples from its slots, put in ascending sample
//              order; a row touched by more from slots and mask (the sample's coefficient for this
//              row is found by binary search in the sample's ascending id list), again in ascending
//              sample order.  So the sums do not depend on the order in which the forward kernel's
//              blocks ran, and no floating-point atomics are used.  Rows touched by many samples are
//              deferred to the end of the block and summed by all its warps.  Adam is then applied
//              to that row only; untouched rows are neither read nor written.  The warp resets the
//              row's count and mask for the next step.
//              The last blocks of the grid update the hidden bias and reduce the batch loss.
//   k_adam_dense : the output layer when every neuron is active (no lists, no masks).
#include "common.cuh"

namespace dslide {

constexpr int UPD_THREADS = 256;
constexpr int UPD_WARPS = UPD_THREADS / 32;
constexpr int HOT_T = 32;      // rows touched by more samples than this are summed by a whole block
constexpr int HOT_MAX = 48;    // deferred rows a block can hold (more: summed by the owning warp)
constexpr unsigned FULL = 0xffffffffu;
// ROW_SLOTS (common.cuh): touches of a row whose (sample, coefficient) the forward kernel stores directly

struct UpdParams {
  float *W1, *mW1, *vW1, *b1, *mb1, *vb1;
  float *W2, *mW2, *vW2, *b2, *mb2, *vb2;
  const float *h, *dh, *act_g, *loss;
  const int32_t *act_cnt, *act_ids;
  const int32_t *row_ptr, *col_idx;
  const float* vals;
  uint32_t *mask1, *mask2, *cnt1, *cnt2;
  const int2 *slots1, *slots2;
  const int32_t *own1, *own2;
  DevState* st;
  float* loss_out;
  int B, H, N, D, Wd, act_stride, dense, parity;
  float lr, beta1, beta2, eps, bc1, bc2;
};

__device__ __forceinline__ void adam1(float& w, float& m, float& v, float g, float b1, float b2, float lr, float eps,
                                      float bc1, float bc2) {
  m = b1 * m + (1.f - b1) * g;
  v = b2 * v + (1.f - b2) * g * g;
  float mhat = m / bc1, vhat = v / bc2;
  w = w - lr * mhat / (sqrtf(vhat) + eps);
}

__device__ __forceinline__ void axpy4(float4& a, float g, const float4 x) {
  a.x = fmaf(g, x.x, a.x); a.y = fmaf(g, x.y, a.y); a.z = fmaf(g, x.z, a.z); a.w = fmaf(g, x.w, a.w);
}

// The pieces of one layer's update: the weight / moment arrays, the rows that multiply the
// coefficients (h for W2, dh for W1), the per-row masks and the bias arrays (W2 only).
struct Side {
  float *W, *M, *V, *bw, *bm, *bv;
  const float* src;
  uint32_t* mask;
  const int2* slots;
  int is_w2;
};

__device__ __forceinline__ Side make_side(const UpdParams& p, bool w2) {
  Side sd;
  sd.W = w2 ? p.W2 : p.W1; sd.M = w2 ? p.mW2 : p.mW1; sd.V = w2 ? p.vW2 : p.vW1;
  sd.bw = p.b2; sd.bm = p.mb2; sd.bv = p.vb2;
  sd.src = w2 ? p.h : p.dh;
  sd.mask = w2 ? p.mask2 : p.mask1;
  sd.slots = w2 ? p.slots2 : p.slots1;
  sd.is_w2 = w2 ? 1 : 0;
  return sd;
}

// Coefficient of (row, sample s): the error of neuron `row` in sample s, or the value of feature
// `row` in sample s.  Both lists are ascending, so a binary search finds it.
__device__ __forceinline__ float find_coef(const UpdParams& p, const Side& sd, const int* sm_rowptr, int row, int s) {
  if (sd.is_w2) {
    const int32_t* ids = p.act_ids + (size_t)s * p.act_stride;
    const int n = p.act_cnt[s];
    int lo = 0, hi = n;
    while (lo < hi) { int mid = (lo + hi) >> 1; if (__ldg(ids + mid) < row) lo = mid + 1; else hi = mid; }
    return (lo < n && __ldg(ids + lo) == row) ? __ldg(p.act_g + (size_t)s * p.act_stride + lo) : 0.f;
  }
  int lo = sm_rowptr[s];
  const int end = sm_rowptr[s + 1];
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
__device__ __forceinline__ void sum_masked(const UpdParams& p, const Side& sd, const int* sm_rowptr, int row,
                                           int slot_s, int w0, int w1, int* scr, float4 (&acc)[NCH], float& csum,
                                           int H, int H4, int lane) {
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
        const float g_mine = lane < fill ? find_coef(p, sd, sm_rowptr, row, s_mine) : 0.f;
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
    const float g_mine = lane < fill ? find_coef(p, sd, sm_rowptr, row, s_mine) : 0.f;
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

template <int NCH>
__device__ __forceinline__ void adam_store(const UpdParams& p, const Side& sd, size_t row, float4 (&w)[NCH],
                                           float4 (&m)[NCH], float4 (&v)[NCH], const float4 (&g)[NCH], int H, int H4,
                                           int lane) {
  float4* w4 = reinterpret_cast<float4*>(sd.W + row * H);
  float4* m4 = reinterpret_cast<float4*>(sd.M + row * H);
  float4* v4 = reinterpret_cast<float4*>(sd.V + row * H);
#pragma unroll
  for (int q = 0; q < NCH; ++q) {
    int c = lane + q * 32;
    if (c < H4) {
      adam1(w[q].x, m[q].x, v[q].x, g[q].x, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
      adam1(w[q].y, m[q].y, v[q].y, g[q].y, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
      adam1(w[q].z, m[q].z, v[q].z, g[q].z, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
      adam1(w[q].w, m[q].w, v[q].w, g[q].w, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
      w4[c] = w[q]; m4[c] = m[q]; v4[c] = v[q];
    }
  }
}

__device__ __forceinline__ void adam_bias(const UpdParams& p, const Side& sd, int row, float g) {
  float w = sd.bw[row], m = sd.bm[row], v = sd.bv[row];
  adam1(w, m, v, g, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
  sd.bw[row] = w; sd.bm[row] = m; sd.bv[row] = v;
}

// The hidden bias (dense gradient, summed over the samples in eight fixed slices) and, in the first
// of these blocks, the mean loss and the step statistics.
__device__ void aux_block(const UpdParams& p, int a, float* sm_part) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, B = p.B;
  const int k = a * 32 + lane;
  const int per = (B + UPD_WARPS - 1) / UPD_WARPS;
  const int s0 = warp * per, s1 = min(B, s0 + per);
  float g = 0.f;
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
  __syncthreads();
  if (warp == 0 && k < H) {
    float tot = 0.f;
    for (int w = 0; w < UPD_WARPS; ++w) tot += sm_part[w * 32 + lane];
    float w = p.b1[k], m = p.mb1[k], v = p.vb1[k];
    adam1(w, m, v, tot, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
    p.b1[k] = w; p.mb1[k] = m; p.vb1[k] = v;
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
    const int q = p.parity, o = q ^ 1;
    st->last[0] = st->acc[q][0]; st->last[1] = st->acc[q][1]; st->last[2] = st->acc[q][2];
    st->cum[0] += 1ull; st->cum[1] += st->acc[q][0]; st->cum[4] += st->acc[q][1]; st->cum[5] += st->acc[q][2];
    if (p.dense) st->cum[2] += (unsigned long long)p.N;
    // the other parity's slots are the next step's: start them at zero
    st->acc[o][0] = 0ull; st->acc[o][1] = 0ull; st->acc[o][2] = 0ull;
    st->cum[3] += (unsigned long long)st->n_own[q][1];
    if (!p.dense) st->cum[2] += (unsigned long long)st->n_own[q][0];
    st->n_own[o][0] = 0u; st->n_own[o][1] = 0u;
  }
}

template <int NCH, int G>
__global__ void __launch_bounds__(UPD_THREADS, (NCH <= 2 ? 2 : 1)) k_update(const UpdParams p) {
  extern __shared__ __align__(16) unsigned char upd_smem[];
  int* sm_rowptr = reinterpret_cast<int*>(upd_smem);                               // [B + 1]
  float* sm_part = reinterpret_cast<float*>(upd_smem + (((size_t)p.B + 1 + 3) & ~(size_t)3) * 4);   // [UPD_WARPS][H + 32]
  __shared__ int hot_list[HOT_MAX];
  __shared__ int hot_n;
  __shared__ int scratch[UPD_WARPS][64];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, B = p.B;
  const int naux = (H + 31) >> 5;
  const int nwork = (int)gridDim.x - naux;
  if ((int)blockIdx.x >= nwork) { aux_block(p, (int)blockIdx.x - nwork, sm_part); return; }

  for (int i = tid; i <= B; i += UPD_THREADS) sm_rowptr[i] = p.row_ptr[i];
  if (tid == 0) hot_n = 0;
  __syncthreads();

  const int n2 = p.dense ? 0 : (int)p.st->n_own[p.parity][0];
  const int n1 = (int)p.st->n_own[p.parity][1];
  const int nrows = n2 + n1;
  const int nwB = (B + 31) >> 5;
  // The concatenated lists (rows of W2, then rows of W1) are dealt out row by row: consecutive rows go to
  // different blocks, because rows touched by many samples tend to sit next to each other in the lists.
  const int nwarps = nwork * UPD_WARPS;
  const int gw = warp * nwork + blockIdx.x;
  const int mine_n = gw < nrows ? (nrows - gw + nwarps - 1) / nwarps : 0;     // rows gw, gw + nwarps, ...

  for (int cb = 0; cb < mine_n; cb += 32) {
    // ids of up to 32 rows of this warp's share, one per lane
    int myrow = 0, myidx = 0;
    if (cb + lane < mine_n) {
      myidx = gw + (cb + lane) * nwarps;
      myrow = myidx < n2 ? p.own2[myidx] : p.own1[myidx - n2];
    }
    const int cend = min(32, mine_n - cb);
    for (int b0 = 0; b0 < cend; b0 += G) {
      int rr[G], tt[G];
      bool live[G], w2[G];
      int2 sl[G];
      float4 w[G][NCH], m[G][NCH], v[G][NCH], x[G][NCH];
#pragma unroll
      for (int q = 0; q < G; ++q) {
        live[q] = b0 + q < cend;
        w2[q] = __shfl_sync(FULL, myidx, live[q] ? b0 + q : 0) < n2;
        rr[q] = __shfl_sync(FULL, myrow, live[q] ? b0 + q : 0);
        tt[q] = 0;
        sl[q] = make_int2(0x7fffffff, 0);
        if (live[q]) {
          const Side sd = make_side(p, w2[q]);
          if (lane == 0) tt[q] = (int)(w2[q] ? p.cnt2 : p.cnt1)[rr[q]];     // read and reset by lane 0 only
          if (lane < ROW_SLOTS) sl[q] = sd.slots[(size_t)rr[q] * ROW_SLOTS + lane];
          load_row<NCH>(sd.W, (size_t)rr[q], H, H4, lane, w[q]);
          load_row<NCH>(sd.M, (size_t)rr[q], H, H4, lane, m[q]);
          load_row<NCH>(sd.V, (size_t)rr[q], H, H4, lane, v[q]);
        }
      }
      // second level: the one sample's row for rows touched once; counts are reset for the next step
#pragma unroll
      for (int q = 0; q < G; ++q)
        if (live[q]) {
          const Side sd = make_side(p, w2[q]);
          if (lane == 0) (w2[q] ? p.cnt2 : p.cnt1)[rr[q]] = 0u;
          tt[q] = __shfl_sync(FULL, tt[q], 0);
          const int s0 = __shfl_sync(FULL, sl[q].x, 0);
          if (tt[q] == 1) load_row<NCH>(sd.src, (size_t)s0, H, H4, lane, x[q]);
        }
#pragma unroll
      for (int q = 0; q < G; ++q)
        if (live[q]) {
          const Side sd = make_side(p, w2[q]);
          float4 acc[NCH];
#pragma unroll
          for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          float csum = 0.f;
          bool defer = false;
          if (tt[q] == 1) {
            const float g0 = __int_as_float(__shfl_sync(FULL, sl[q].y, 0));
#pragma unroll
            for (int u = 0; u < NCH; ++u) axpy4(acc[u], g0, x[q][u]);
            csum = g0;
          } else if (tt[q] <= ROW_SLOTS) {
            sum_slots<NCH>(sd, sl[q], tt[q], scratch[warp], acc, csum, H, H4, lane);
          } else {
            if (tt[q] > HOT_T) {
              int slot = 0;
              if (lane == 0) slot = atomicAdd(&hot_n, 1);
              slot = __shfl_sync(FULL, slot, 0);
              if (slot < HOT_MAX) {
                if (lane == 0) hot_list[slot] = w2[q] ? rr[q] : ~rr[q];
                defer = true;
              }
            }
            if (!defer) sum_masked<NCH>(p, sd, sm_rowptr, rr[q], sl[q].x, 0, nwB, scratch[warp], acc, csum, H, H4, lane);
          }
          if (!defer) {
            adam_store<NCH>(p, sd, (size_t)rr[q], w[q], m[q], v[q], acc, H, H4, lane);
            if (w2[q] && lane == 0) adam_bias(p, sd, rr[q], csum);
          }
        }
    }
  }

  // ---- rows touched by many samples: every warp sums a slice of the row's mask, slices added in order ----
  __syncthreads();
  const int nh = hot_n < HOT_MAX ? hot_n : HOT_MAX;
  const int ld = H + 32;
  for (int qh = 0; qh < nh; ++qh) {
    const int code = hot_list[qh];
    const bool w2 = code >= 0;
    const int row = w2 ? code : ~code;
    const Side sd = make_side(p, w2);
    const int per_w = (nwB + UPD_WARPS - 1) / UPD_WARPS;
    const int w0 = min(nwB, warp * per_w), w1 = min(nwB, w0 + per_w);
    float4 acc[NCH];
#pragma unroll
    for (int u = 0; u < NCH; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    float csum = 0.f;
    int slot_s = 0x7fffffff;
    if (lane < ROW_SLOTS) slot_s = sd.slots[(size_t)row * ROW_SLOTS + lane].x;
    sum_masked<NCH>(p, sd, sm_rowptr, row, slot_s, w0, w1, scratch[warp], acc, csum, H, H4, lane);
    float4* mine = reinterpret_cast<float4*>(sm_part + (size_t)warp * ld);
#pragma unroll
    for (int u = 0; u < NCH; ++u) {
      int cidx = lane + u * 32;
      if (cidx < H4) mine[cidx] = acc[u];
    }
    if (lane == 0) sm_part[(size_t)warp * ld + H] = csum;
    __syncthreads();
    for (int k = tid; k < H; k += UPD_THREADS) {
      float gsum = 0.f;
      for (int w = 0; w < UPD_WARPS; ++w) gsum += sm_part[(size_t)w * ld + k];
      const size_t e = (size_t)row * H + k;
      float wv = sd.W[e], mv = sd.M[e], vv = sd.V[e];
      adam1(wv, mv, vv, gsum, p.beta1, p.beta2, p.lr, p.eps, p.bc1, p.bc2);
      sd.W[e] = wv; sd.M[e] = mv; sd.V[e] = vv;
    }
    if (w2 && tid == 0) {
      float cs = 0.f;
      for (int w = 0; w < UPD_WARPS; ++w) cs += sm_part[(size_t)w * ld + H];
      adam_bias(p, sd, row, cs);
    }
    __syncthreads();
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
    if (lane == 0) adam_bias(p, sd, j, csum);
  }
}

template <int NCH, int G>
static cudaError_t launch_k_update(Ctx* c, const UpdParams& p, int smem) {
  cudaError_t e = cudaSuccess;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(k_update<NCH, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  const int naux = (c->H + 31) / 32;
  LaunchScope ls(c, KID_ADAM);
  k_update<NCH, G><<<c->num_sms * (NCH <= 2 ? 2 : 1) + naux, UPD_THREADS, smem, c->stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_update(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                          float* loss_out) {
  UpdParams p;
  p.W1 = c->W1; p.mW1 = c->mW1; p.vW1 = c->vW1; p.b1 = c->b1; p.mb1 = c->mb1; p.vb1 = c->vb1;
  p.W2 = c->W2; p.mW2 = c->mW2; p.vW2 = c->vW2; p.b2 = c->b2; p.mb2 = c->mb2; p.vb2 = c->vb2;
  p.h = c->h; p.dh = c->dh; p.act_g = c->act_g; p.loss = c->loss; p.act_cnt = c->act_cnt; p.act_ids = c->act_ids;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.vals = vals;
  p.mask1 = c->mask1; p.mask2 = c->mask2; p.cnt1 = c->cnt1; p.cnt2 = c->cnt2;
  p.slots1 = c->slots1; p.slots2 = c->slots2; p.own1 = c->own1; p.own2 = c->own2;
  p.st = c->dstate; p.loss_out = loss_out;
  p.B = batch; p.H = c->H; p.N = c->N; p.D = c->D; p.Wd = c->Wd; p.act_stride = c->act_stride; p.dense = c->dense;
  p.parity = (int)(c->t_host & 1);
  p.lr = c->cfg.lr; p.beta1 = c->cfg.beta1; p.beta2 = c->cfg.beta2; p.eps = c->cfg.eps;
  // bias corrections of Adam with the global step count (the step being taken is t + 1)
  const double t = (double)(c->t_host + 1);
  p.bc1 = (float)(1.0 - pow((double)c->cfg.beta1, t));
  p.bc2 = (float)(1.0 - pow((double)c->cfg.beta2, t));

  if (c->dense) {
    LaunchScope ls(c, KID_ADAM_DENSE);
    k_adam_dense<<<c->num_sms * 4, UPD_THREADS, 0, c->stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int smem = (((batch + 1 + 3) & ~3) + UPD_WARPS * (c->H + 32)) * 4;
  const int nch = (c->H / 4 + 31) / 32;
  if (nch <= 1) return launch_k_update<1, 4>(c, p, smem);
  if (nch <= 2) return launch_k_update<2, 2>(c, p, smem);
  if (nch <= 4) return launch_k_update<4, 1>(c, p, smem);
  return launch_k_update<8, 1>(c, p, smem);
}

}  // namespace dslide
