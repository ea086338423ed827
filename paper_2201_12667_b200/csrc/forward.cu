// Per-sample forward kernel of the SLIDE step: one thread block per sample runs
//   hidden layer (Section 3.6, feed forward of the first type: sparse input)
//   -> L bucket codes of the hidden activation (SimHash or DWTA, Section 4.1)
//   -> bucket lookup, union over the tables plus the labels (Section 2.1, Fig. 1)
//   -> logits over the active set only (feed forward of the second type)
//   -> softmax, loss and errors over that ragged set (Algorithm 1 "Compute Errors")
//   -> error back-propagated to the hidden layer (Section 2.1, back-propagation stage)
// and records, for the update kernels, which rows of W2 and W1 the sample touches.
// The same kernel in predict mode stops after the logits and selects the top k.
#include "common.cuh"

namespace dslide {

constexpr int FWD_THREADS = 256;
constexpr int FWD_WARPS = FWD_THREADS / 32;
constexpr int MAX_HCHUNK = 8;   // float4 chunks per lane: H <= 4 * 32 * 8 = 1024

struct FwdParams {
  const float *W1, *b1, *W2, *b2;
  const int32_t *hash_idx, *hash_sign, *bucket_off, *bucket_ids;
  const int32_t *row_ptr, *col_idx;
  const float* vals;
  const int32_t *label_ptr, *labels;
  float *h, *dh, *loss;
  uint32_t* codes;
  int32_t *act_cnt, *act_ids;
  float *act_z, *act_p, *act_g;
  uint32_t *mask1, *mask2, *cnt1, *cnt2;
  int2 *slots1, *slots2;
  int32_t *own1, *own2, *hot_rows, *med_rows;
  DevState* st;
  int32_t* out_ids;
  float* out_scores;
  long long nb;
  int B, D, H, N, K, L, KL, family, lg_bin, fn_len, cap;
  int act_stride, Wd, dense, dedup_mode, max_labels, sort_cap, topk, parity;
  int off_dh, off_code, off_part, off_misc, off_lab, off_tbase, off_topk, off_dedup;
};

__device__ __forceinline__ void set_status(DevState* st, int code) { atomicCAS(&st->status, 0, code); }

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

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
// sh needs FWD_WARPS + 1 ints.  Ends with a barrier, so sh may be reused afterwards.
__device__ __forceinline__ int block_excl_scan(int v, int* sh, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, incl, d);
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
  for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int w = 1; w < FWD_WARPS; ++w) r = fmaxf(r, sh[w]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float block_sum(float v, float* sh) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
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

template <int MODE>   // 0 = training step, 1 = predict top-k
__global__ void __launch_bounds__(FWD_THREADS) k_forward(const FwdParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  float* sh_h = reinterpret_cast<float*>(smem);
  float* sh_dh = reinterpret_cast<float*>(smem + p.off_dh);          // [FWD_WARPS][H]
  uint32_t* sh_code = reinterpret_cast<uint32_t*>(smem + p.off_code);
  unsigned char* sh_part = smem + p.off_part;
  int* sh_misc = reinterpret_cast<int*>(smem + p.off_misc);          // 32 ints
  float* sh_red = reinterpret_cast<float*>(sh_misc + 16);
  int* sh_lab = reinterpret_cast<int*>(smem + p.off_lab);            // [max_labels]
  int* sh_tbase = reinterpret_cast<int*>(smem + p.off_tbase);        // [L + 1]
  uint32_t* sh_dd = reinterpret_cast<uint32_t*>(smem + p.off_dedup);

  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, N = p.N;
  const int rbeg = p.row_ptr[s], rend = p.row_ptr[s + 1];
  const int nnz = rend - rbeg;
  int lbeg = 0, nlab = 0;
  if (MODE == 0) { lbeg = p.label_ptr[s]; nlab = p.label_ptr[s + 1] - lbeg; }

  // ---- input checks: ids in range, columns ascending, label list within the maximum ----
  int bad = 0;
  if (nnz < 0 || nlab < 0) bad = DSLIDE_ERR_BAD_INDEX;
  else {
    for (int i = tid; i < nnz; i += FWD_THREADS) {
      int c = p.col_idx[rbeg + i];
      if (c < 0 || c >= p.D || (i > 0 && p.col_idx[rbeg + i - 1] >= c)) bad = DSLIDE_ERR_BAD_INDEX;
    }
    if (MODE == 0) {
      for (int i = tid; i < nlab; i += FWD_THREADS) {
        int y = p.labels[lbeg + i];
        if (y < 0 || y >= N) bad = DSLIDE_ERR_BAD_INDEX;
      }
      if (nlab > p.max_labels) bad = DSLIDE_ERR_OVERFLOW;
    }
  }
  if (tid == 0) sh_misc[24] = 0;               // bucket entries fetched by this sample
  bad = __syncthreads_or(bad);
  if (bad) {
    // The sample is skipped: no loss, no gradient, nothing touched.
    if (MODE == 0) {
      for (int k = tid; k < H; k += FWD_THREADS) { p.h[(size_t)s * H + k] = 0.f; p.dh[(size_t)s * H + k] = 0.f; }
      if (tid == 0) { p.act_cnt[s] = 0; p.loss[s] = 0.f; }
    } else {
      for (int q = tid; q < p.topk; q += FWD_THREADS) {
        p.out_ids[(size_t)s * p.topk + q] = -1;
        p.out_scores[(size_t)s * p.topk + q] = -INFINITY;
      }
    }
    if (tid == 0) {
      int code = DSLIDE_ERR_BAD_INDEX;
      if (MODE == 0 && nnz >= 0 && nlab > p.max_labels) code = DSLIDE_ERR_OVERFLOW;
      set_status(p.st, code);
    }
    return;
  }

  // ---- hidden layer: bias, then one fused multiply-add per nonzero in stored order, ReLU ----
  for (int k = tid; k < H; k += FWD_THREADS) {
    float acc = p.b1[k];
    int i = rbeg;
    for (; i + 4 <= rend; i += 4) {
      int c0 = __ldg(p.col_idx + i), c1 = __ldg(p.col_idx + i + 1), c2 = __ldg(p.col_idx + i + 2), c3 = __ldg(p.col_idx + i + 3);
      float x0 = __ldg(p.vals + i), x1 = __ldg(p.vals + i + 1), x2 = __ldg(p.vals + i + 2), x3 = __ldg(p.vals + i + 3);
      float w0 = __ldg(p.W1 + (size_t)c0 * H + k), w1 = __ldg(p.W1 + (size_t)c1 * H + k);
      float w2 = __ldg(p.W1 + (size_t)c2 * H + k), w3 = __ldg(p.W1 + (size_t)c3 * H + k);
      acc = __fmaf_rn(x0, w0, acc);
      acc = __fmaf_rn(x1, w1, acc);
      acc = __fmaf_rn(x2, w2, acc);
      acc = __fmaf_rn(x3, w3, acc);
    }
    for (; i < rend; ++i) acc = __fmaf_rn(__ldg(p.vals + i), __ldg(p.W1 + (size_t)__ldg(p.col_idx + i) * H + k), acc);
    float hv = acc > 0.f ? acc : 0.f;
    sh_h[k] = hv;
    if (MODE == 0) p.h[(size_t)s * H + k] = hv;
  }
  __syncthreads();

  const bool dense = p.dense != 0;
  int na = N;
  int32_t* ids = p.act_ids + (size_t)s * p.act_stride;

  if (!dense) {
    // ---- bucket codes of the hidden activation ----
    for (int f = tid; f < p.KL; f += FWD_THREADS) {
      const int32_t* ix = p.hash_idx + (size_t)f * p.fn_len;
      if (p.family == DSLIDE_SIMHASH) {
        const int32_t* sg = p.hash_sign + (size_t)f * p.fn_len;
        float sum = 0.f;
        for (int i = 0; i < p.fn_len; ++i) {
          float x = sh_h[__ldg(ix + i)];
          sum = __fadd_rn(sum, __ldg(sg + i) > 0 ? x : -x);
        }
        sh_part[f] = sum >= 0.f ? 1 : 0;
      } else {
        int best = 0;
        float bv = sh_h[__ldg(ix)];
        for (int i = 1; i < p.fn_len; ++i) {
          float v = sh_h[__ldg(ix + i)];
          if (v > bv) { bv = v; best = i; }       // strict: the lowest position wins ties
        }
        sh_part[f] = (unsigned char)best;
      }
    }
    __syncthreads();
    const int shift = p.family == DSLIDE_SIMHASH ? 1 : p.lg_bin;
    for (int t = tid; t < p.L; t += FWD_THREADS) {
      uint32_t code = 0;
      for (int k = 0; k < p.K; ++k) code |= (uint32_t)sh_part[t * p.K + k] << (k * shift);
      sh_code[t] = code;
      if (MODE == 0) p.codes[(size_t)s * p.L + t] = code;
    }
    __syncthreads();

    // ---- lookup, union over the tables, labels, duplicates removed, ascending ids ----
    int total = 0;
    if (p.dedup_mode == 1) {
      const int nwords = (N + 31) >> 5;
      for (int w = tid; w < nwords; w += FWD_THREADS) sh_dd[w] = 0u;
      __syncthreads();
      for (int t = warp; t < p.L; t += FWD_WARPS) {
        const int32_t* off = p.bucket_off + (size_t)t * (size_t)(p.nb + 1);
        const int beg = __ldg(off + sh_code[t]);
        int cnt = __ldg(off + sh_code[t] + 1) - beg;
        cnt = cnt < p.cap ? cnt : p.cap;
        const int32_t* bid = p.bucket_ids + (size_t)t * N + beg;
        for (int i = lane; i < cnt; i += 32) {
          int j = __ldg(bid + i);
          atomicOr(&sh_dd[j >> 5], 1u << (j & 31));
        }
        if (lane == 0) atomicAdd(&sh_misc[24], cnt);
      }
      if (MODE == 0)
        for (int i = tid; i < nlab; i += FWD_THREADS) {
          int y = p.labels[lbeg + i];
          atomicOr(&sh_dd[y >> 5], 1u << (y & 31));
        }
      __syncthreads();
      const int chunk = (nwords + FWD_THREADS - 1) / FWD_THREADS;
      const int wbeg = tid * chunk, wend = min(nwords, wbeg + chunk);
      int cnt = 0;
      for (int w = wbeg; w < wend; ++w) cnt += __popc(sh_dd[w]);
      int pos = block_excl_scan(cnt, sh_misc, &total);
      if (total <= p.act_stride) {
        for (int w = wbeg; w < wend; ++w) {
          uint32_t bits = sh_dd[w];
          while (bits) {
            int b = __ffs(bits) - 1;
            ids[pos++] = (w << 5) + b;
            bits &= bits - 1;
          }
        }
      }
    } else {
      // sort path: gather all candidates, bitonic sort, keep the first of each run
      for (int t = tid; t < p.L; t += FWD_THREADS) {
        const int32_t* off = p.bucket_off + (size_t)t * (size_t)(p.nb + 1);
        int cnt = __ldg(off + sh_code[t] + 1) - __ldg(off + sh_code[t]);
        sh_tbase[t] = cnt < p.cap ? cnt : p.cap;
      }
      __syncthreads();
      if (tid == 0) {
        int run = 0;
        for (int t = 0; t < p.L; ++t) { int c = sh_tbase[t]; sh_tbase[t] = run; run += c; }
        sh_tbase[p.L] = run;
      }
      __syncthreads();
      const int ncand = sh_tbase[p.L] + nlab;     // <= L*cap + max_labels <= sort_cap
      if (tid == 0) sh_misc[24] = sh_tbase[p.L];
      int n2 = 1;
      while (n2 < ncand) n2 <<= 1;
      for (int t = warp; t < p.L; t += FWD_WARPS) {
        const int32_t* off = p.bucket_off + (size_t)t * (size_t)(p.nb + 1);
        const int beg = __ldg(off + sh_code[t]);
        const int cnt = sh_tbase[t + 1] - sh_tbase[t];
        const int32_t* bid = p.bucket_ids + (size_t)t * N + beg;
        for (int i = lane; i < cnt; i += 32) sh_dd[sh_tbase[t] + i] = (uint32_t)__ldg(bid + i);
      }
      if (MODE == 0)
        for (int i = tid; i < nlab; i += FWD_THREADS) sh_dd[sh_tbase[p.L] + i] = (uint32_t)p.labels[lbeg + i];
      for (int i = ncand + tid; i < n2; i += FWD_THREADS) sh_dd[i] = 0x7fffffffu;
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
          if (a != 0x7fffffffu && (i == 0 || sh_dd[i - 1] != a)) ids[pos++] = (int)a;
        }
      }
    }
    if (total > p.act_stride) {      // uniform over the block
      if (MODE == 0) {
        for (int k = tid; k < H; k += FWD_THREADS) { p.h[(size_t)s * H + k] = 0.f; p.dh[(size_t)s * H + k] = 0.f; }
        if (tid == 0) { p.act_cnt[s] = 0; p.loss[s] = 0.f; }
      } else {
        for (int q = tid; q < p.topk; q += FWD_THREADS) {
          p.out_ids[(size_t)s * p.topk + q] = -1;
          p.out_scores[(size_t)s * p.topk + q] = -INFINITY;
        }
      }
      if (tid == 0) set_status(p.st, DSLIDE_ERR_OVERFLOW);
      return;
    }
    na = total;
    __syncthreads();
  }
  if (MODE == 0 && tid == 0) p.act_cnt[s] = na;

  // ---- logits over the active set: one warp per neuron, four neurons in flight ----
  float* z = p.act_z + (size_t)s * p.act_stride;
  float* tk_z = reinterpret_cast<float*>(smem + p.off_topk);          // predict: [FWD_WARPS][topk]
  int* tk_id = reinterpret_cast<int*>(tk_z + FWD_WARPS * p.topk);
  int tk_cnt = 0;                                                     // used by lane 0
  const float4* sh_h4 = reinterpret_cast<const float4*>(sh_h);
  for (int a0 = warp * 4; a0 < na; a0 += FWD_WARPS * 4) {
    int j[4];
    float acc[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      int a = a0 + r;
      j[r] = a < na ? (dense ? a : ids[a]) : -1;
      acc[r] = 0.f;
    }
    for (int c = lane; c < H4; c += 32) {
      float4 x = sh_h4[c];
      float4 w[4];
#pragma unroll
      for (int r = 0; r < 4; ++r)
        w[r] = j[r] >= 0 ? __ldg(reinterpret_cast<const float4*>(p.W2 + (size_t)j[r] * H) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        acc[r] = fmaf(w[r].x, x.x, acc[r]);
        acc[r] = fmaf(w[r].y, x.y, acc[r]);
        acc[r] = fmaf(w[r].z, x.z, acc[r]);
        acc[r] = fmaf(w[r].w, x.w, acc[r]);
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], d);
    }
    if (MODE == 0) {
#pragma unroll
      for (int r = 0; r < 4; ++r)
        if (lane == r && j[r] >= 0) z[a0 + r] = __ldg(p.b2 + j[r]) + acc[r];
    } else if (lane == 0) {
      float* lz = tk_z + warp * p.topk;
      int* li = tk_id + warp * p.topk;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        if (j[r] < 0) continue;
        float zv = __ldg(p.b2 + j[r]) + acc[r];
        if (tk_cnt < p.topk || topk_better(zv, j[r], lz[tk_cnt - 1], li[tk_cnt - 1])) {
          int q = tk_cnt < p.topk ? tk_cnt++ : p.topk - 1;
          while (q > 0 && topk_better(zv, j[r], lz[q - 1], li[q - 1])) { lz[q] = lz[q - 1]; li[q] = li[q - 1]; --q; }
          lz[q] = zv; li[q] = j[r];
        }
      }
    }
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

  // ---- positions of the sample's distinct labels inside the active set ----
  for (int i = tid; i < nlab; i += FWD_THREADS) {
    int y = p.labels[lbeg + i];
    bool first = true;
    for (int q = 0; q < i; ++q) first = first && (p.labels[lbeg + q] != y);
    int pos = y;
    if (!dense) {
      int lo = 0, hi = na;
      while (lo < hi) { int mid = (lo + hi) >> 1; if (ids[mid] < y) lo = mid + 1; else hi = mid; }
      pos = lo;
    }
    sh_lab[i] = first ? pos : -1;
  }
  __syncthreads();

  // ---- softmax over the ragged active set, loss, errors ----
  float* pr = p.act_p + (size_t)s * p.act_stride;
  float* g = p.act_g + (size_t)s * p.act_stride;
  float m = -INFINITY;
  for (int a = tid; a < na; a += FWD_THREADS) m = fmaxf(m, z[a]);
  const float M = block_max(m, sh_red);
  float e = 0.f;
  for (int a = tid; a < na; a += FWD_THREADS) e += expf(z[a] - M);
  const float E = block_sum(e, sh_red);
  const float fB = (float)p.B;
  for (int a = tid; a < na; a += FWD_THREADS) {
    float pa = expf(z[a] - M) / E;
    pr[a] = pa;
    g[a] = pa / fB;
  }
  __syncthreads();
  if (tid == 0) {
    int ny = 0;
    for (int i = 0; i < nlab; ++i) ny += sh_lab[i] >= 0 ? 1 : 0;
    float sum = 0.f;
    const float logE = logf(E);
    for (int i = 0; i < nlab; ++i)
      if (sh_lab[i] >= 0) sum += z[sh_lab[i]] - M - logE;
    p.loss[s] = ny > 0 ? -sum / (float)ny : 0.f;
    sh_misc[0] = ny;
  }
  __syncthreads();
  {
    const int ny = sh_misc[0];
    for (int i = tid; i < nlab; i += FWD_THREADS)
      if (sh_lab[i] >= 0) g[sh_lab[i]] = (pr[sh_lab[i]] - 1.f / (float)ny) / fB;
  }
  __syncthreads();

  // ---- error at the hidden layer: dh = [h > 0] * sum_a g_a W2[j_a, :] (weights before the update) ----
  {
    float4 acc[MAX_HCHUNK];
#pragma unroll
    for (int q = 0; q < MAX_HCHUNK; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int a = warp; a < na; a += FWD_WARPS) {
      const int jj = dense ? a : ids[a];
      const float ga = g[a];
      const float4* row = reinterpret_cast<const float4*>(p.W2 + (size_t)jj * H);
#pragma unroll
      for (int q = 0; q < MAX_HCHUNK; ++q) {
        int c = lane + q * 32;
        if (c < H4) {
          float4 w = __ldg(row + c);
          acc[q].x = fmaf(ga, w.x, acc[q].x);
          acc[q].y = fmaf(ga, w.y, acc[q].y);
          acc[q].z = fmaf(ga, w.z, acc[q].z);
          acc[q].w = fmaf(ga, w.w, acc[q].w);
        }
      }
    }
    float4* mine = reinterpret_cast<float4*>(sh_dh + (size_t)warp * H);
#pragma unroll
    for (int q = 0; q < MAX_HCHUNK; ++q) {
      int c = lane + q * 32;
      if (c < H4) mine[c] = acc[q];
    }
  }
  __syncthreads();
  for (int k = tid; k < H; k += FWD_THREADS) {
    float v = 0.f;
    for (int w = 0; w < FWD_WARPS; ++w) v += sh_dh[(size_t)w * H + k];
    p.dh[(size_t)s * H + k] = sh_h[k] > 0.f ? v : 0.f;
  }

  // ---- hand the sample's touches to the update kernel.  Per touched row: a count of the touching samples;
  //      for the row's first ROW_SLOTS touches the (sample, coefficient) pair itself, else the bit of this
  //      sample in the row's mask.  The sample that touches a row first also enters it in the list of
  //      distinct rows (positions handed out per warp). ----
  const uint32_t sbit = 1u << (s & 31);
  const int sword = s >> 5;
  const unsigned lt = (1u << lane) - 1u;
  if (!dense)
    for (int a0 = 0; a0 < na; a0 += FWD_THREADS) {
      const int a = a0 + tid;
      bool first = false;
      int jj = 0;
      if (a < na) {
        jj = ids[a];
        const unsigned nth = atomicAdd(p.cnt2 + jj, 1u) & CNT_MASK;
        if (nth < (unsigned)ROW_SLOTS) p.slots2[(size_t)jj * ROW_SLOTS + nth] = make_int2(s, __float_as_int(g[a]));
        else atomicOr(p.mask2 + (size_t)jj * p.Wd + sword, sbit);
        first = nth == 0u;
        list_row(p, p.cnt2 + jj, jj, nth);
      }
      const unsigned fm = __ballot_sync(0xffffffffu, first);
      if (fm) {
        unsigned base = 0;
        if (lane == 0) base = atomicAdd(&p.st->n_own[p.parity][0], (unsigned)__popc(fm));
        base = __shfl_sync(0xffffffffu, base, 0);
        if (first) p.own2[base + __popc(fm & lt)] = jj;
      }
    }
  for (int i0 = 0; i0 < nnz; i0 += FWD_THREADS) {
    const int i = i0 + tid;
    bool first = false;
    int c = 0;
    if (i < nnz) {
      c = p.col_idx[rbeg + i];
      const unsigned nth = atomicAdd(p.cnt1 + c, 1u) & CNT_MASK;
      if (nth < (unsigned)ROW_SLOTS) p.slots1[(size_t)c * ROW_SLOTS + nth] = make_int2(s, __float_as_int(p.vals[rbeg + i]));
      else atomicOr(p.mask1 + (size_t)c * p.Wd + sword, sbit);
      first = nth == 0u;
      list_row(p, p.cnt1 + c, ~c, nth);
    }
    const unsigned fm = __ballot_sync(0xffffffffu, first);
    if (fm) {
      unsigned base = 0;
      if (lane == 0) base = atomicAdd(&p.st->n_own[p.parity][1], (unsigned)__popc(fm));
      base = __shfl_sync(0xffffffffu, base, 0);
      if (first) p.own1[base + __popc(fm & lt)] = c;
    }
  }
  if (tid == 0) {
    atomicAdd(&p.st->acc[p.parity][0], (unsigned long long)na);
    atomicAdd(&p.st->acc[p.parity][1], (unsigned long long)nnz);
    atomicAdd(&p.st->acc[p.parity][2], (unsigned long long)sh_misc[24]);
  }
}

// ---------------------------------------------------------------------------
// Host side: shared-memory layout and launches
// ---------------------------------------------------------------------------
static int align16(int x) { return (x + 15) & ~15; }

struct FwdLayout { int off_dh, off_code, off_part, off_misc, off_lab, off_tbase, off_topk, off_dedup, fixed_bytes; };

static FwdLayout fwd_layout(const Ctx* c) {
  FwdLayout l;
  int o = align16(c->H * 4);
  l.off_dh = o;      o = align16(o + FWD_WARPS * c->H * 4);
  l.off_code = o;    o = align16(o + c->L * 4);
  l.off_part = o;    o = align16(o + c->KL);
  l.off_misc = o;    o = align16(o + 32 * 4);
  l.off_lab = o;     o = align16(o + (c->cfg.max_labels > 0 ? c->cfg.max_labels : 1) * 4);
  l.off_tbase = o;   o = align16(o + (c->L + 1) * 4);
  l.off_topk = o;    o = align16(o + FWD_WARPS * 64 * 8);
  l.off_dedup = o;
  l.fixed_bytes = o;
  return l;
}

cudaError_t setup_forward(Ctx* c) {
  FwdLayout l = fwd_layout(c);
  const int budget = 227 * 1024 - l.fixed_bytes;
  const int bitmap_bytes = ((c->N + 31) / 32) * 4;
  int64_t worst = (int64_t)c->L * c->cap + c->cfg.max_labels;
  int64_t pow2 = 1;
  while (pow2 < worst) pow2 <<= 1;
  const int64_t sort_bytes = pow2 * 4;
  int mode = c->cfg.dedup_mode;
  if (c->dense) { mode = 1; c->fwd_smem = l.fixed_bytes; c->sort_cap = 0; c->dedup_mode = 1; }
  else {
    if (mode == 0) mode = (bitmap_bytes <= 100 * 1024 || sort_bytes > budget) ? 1 : 2;
    if (mode == 1 && bitmap_bytes > budget) return cudaErrorInvalidValue;
    if (mode == 2 && sort_bytes > budget) return cudaErrorInvalidValue;
    c->dedup_mode = mode;
    c->sort_cap = (int)pow2;
    c->fwd_smem = l.fixed_bytes + (mode == 1 ? bitmap_bytes : (int)sort_bytes);
  }
  cudaError_t e = cudaFuncSetAttribute(k_forward<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_forward<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

static FwdParams make_params(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                             const int32_t* label_ptr, const int32_t* labels) {
  FwdParams p;
  p.W1 = c->W1; p.b1 = c->b1; p.W2 = c->W2; p.b2 = c->b2;
  p.hash_idx = c->hash_idx; p.hash_sign = c->hash_sign; p.bucket_off = c->bucket_off; p.bucket_ids = c->bucket_ids;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.vals = vals; p.label_ptr = label_ptr; p.labels = labels;
  p.h = c->h; p.dh = c->dh; p.loss = c->loss; p.codes = c->codes;
  p.act_cnt = c->act_cnt; p.act_ids = c->act_ids; p.act_z = c->act_z; p.act_p = c->act_p; p.act_g = c->act_g;
  p.mask1 = c->mask1; p.mask2 = c->mask2; p.cnt1 = c->cnt1; p.cnt2 = c->cnt2;
  p.slots1 = c->slots1; p.slots2 = c->slots2;
  p.own1 = c->own1; p.own2 = c->own2; p.hot_rows = c->hot_rows; p.med_rows = c->med_rows; p.parity = (int)(c->t_host & 1);
  p.st = c->dstate; p.out_ids = nullptr; p.out_scores = nullptr;
  p.nb = c->nb;
  p.B = batch; p.D = c->D; p.H = c->H; p.N = c->N; p.K = c->K; p.L = c->L; p.KL = c->KL;
  p.family = c->cfg.hash_family; p.lg_bin = c->lg_bin; p.fn_len = c->fn_len; p.cap = c->cap;
  p.act_stride = c->act_stride; p.Wd = c->Wd; p.dense = c->dense; p.dedup_mode = c->dedup_mode;
  p.max_labels = c->cfg.max_labels; p.sort_cap = c->sort_cap; p.topk = 1;
  FwdLayout l = fwd_layout(c);
  p.off_dh = l.off_dh; p.off_code = l.off_code; p.off_part = l.off_part; p.off_misc = l.off_misc;
  p.off_lab = l.off_lab; p.off_tbase = l.off_tbase; p.off_topk = l.off_topk; p.off_dedup = l.off_dedup;
  return p;
}

cudaError_t launch_forward_train(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                                 const int32_t* label_ptr, const int32_t* labels) {
  FwdParams p = make_params(c, batch, row_ptr, col_idx, vals, label_ptr, labels);
  {
    LaunchScope ls(c, KID_FORWARD);
    k_forward<0><<<batch, FWD_THREADS, c->fwd_smem, c->stream>>>(p);
  }
  return cudaGetLastError();
}

cudaError_t launch_predict(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                           int k, int dense, int32_t* out_ids, float* out_scores) {
  FwdParams p = make_params(c, batch, row_ptr, col_idx, vals, nullptr, nullptr);
  p.topk = k;
  p.out_ids = out_ids;
  p.out_scores = out_scores;
  int smem = c->fwd_smem;
  if (dense) { p.dense = 1; smem = fwd_layout(c).fixed_bytes; }
  {
    LaunchScope ls(c, KID_PREDICT);
    k_forward<1><<<batch, FWD_THREADS, smem, c->stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace dslide
